"""ctypes binding of libemaslice.so — argument marshalling only.

Every step of the path (block tables, gather, attention, migration) runs inside the library; this
module converts Python values to the C ABI of ``include/emaslice.h`` and back. Functions carry the
names of the C entry points. The library must be present: loading fails loudly when it is missing
(there is no fallback of any kind).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libemaslice.so")

OK, EINVAL, ENOSPC, ESTAGING, ESTALE, ECUDA, ETIMEOUT, ESTATE, ESCRATCH, ECAPPED = 0, -1, -2, -3, -4, -5, -6, -7, -8, -9
PREEMPT_OOM, PREEMPT_RECLAIM = 1, 2
TIER_AUTO, TIER_LOCAL, TIER_LENT = 0, 1, 2
FLAG_PROFILE, FLAG_TRACE, FLAG_NULL_DEVICE = 1, 2, 4
FLAG_TEST_WITHHOLD_Q, FLAG_TEST_FAIL_COPY = 8, 16      # test hooks (see include/emaslice.h)
COPY_DEFAULT, COPY_VECTOR, COPY_BULK, COPY_BULK_SHARED = 0, 1, 2, 3
LAYOUT_LAYER_MAJOR, LAYOUT_SLAB_MAJOR, LAYOUT_LAYER_GROUP_MAJOR = 0, 1, 2
TAKE_ALL = 0xFFFFFFFF

EXPORTS = [
    "slice_create", "slice_destroy", "slice_alloc_blocks", "slice_set_seq_len", "slice_free_seq",
    "slice_get_block_table", "slice_get_free_stack", "prefetch_layer", "paged_decode", "slice_reclaim",
    "slice_lend", "slice_append_kv", "slice_writeback_layer", "slice_decode_step", "slice_stats",
    "slice_get_resolved", "slice_layer_times", "slice_copy_blocks", "slice_strerror", "paged_decode_noalloc", "slice_cta_trace",
    "slice_reclaim_preempt", "slice_preempt_seq", "slice_set_preempt_window", "slice_set_time", "slice_preempt_stats",
    "slice_set_peer_used", "slice_schedule_gll",
    "slice_step_begin", "slice_step_submit_q", "slice_step_wait_out", "slice_step_flags", "slice_step_relay",
    "slice_copy_blocks_series",
]


class SliceConfig(C.Structure):
    _fields_ = [
        ("num_layers", C.c_uint32), ("num_kv_heads", C.c_uint32), ("head_dim", C.c_uint32),
        ("block_tokens", C.c_uint32), ("dtype", C.c_uint32), ("local_blocks", C.c_uint32),
        ("lent_blocks", C.c_uint32), ("lent_blocks_physical", C.c_uint32), ("ring_slots", C.c_uint32),
        ("staging_blocks_per_slot", C.c_uint32), ("max_seqs", C.c_uint32), ("max_blocks_per_seq", C.c_uint32),
        ("lent_kind", C.c_uint32), ("flags", C.c_uint32),
        ("local_base", C.c_void_p), ("lent_base", C.c_void_p), ("staging_base", C.c_void_p),
        ("local_layer_stride", C.c_uint64), ("local_block_stride", C.c_uint64),
        ("lent_layer_stride", C.c_uint64), ("lent_block_stride", C.c_uint64),
        ("local_free_order", C.c_void_p), ("lent_free_order", C.c_void_p),
        ("decode_ctas", C.c_uint32), ("copy_ctas", C.c_uint32), ("copy_kind", C.c_uint32),
        ("pipeline_mode", C.c_uint32), ("static_split", C.c_uint32), ("claim_blocks", C.c_uint32),
        ("steal_floor", C.c_uint32), ("prefetch_priority", C.c_uint32),
        ("slab_blocks", C.c_uint32), ("layer_group", C.c_uint32), ("layout", C.c_uint32),
        ("split_layer", C.c_uint32), ("swap_out", C.c_uint32),
    ]


class SliceStats(C.Structure):
    _fields_ = [
        ("local_used", C.c_uint32), ("local_free", C.c_uint32), ("lent_used", C.c_uint32),
        ("lent_free", C.c_uint32), ("lent_capacity", C.c_uint32), ("num_seqs", C.c_uint32),
        ("prefetch_calls", C.c_uint64), ("prefetched_blocks", C.c_uint64), ("prefetched_bytes", C.c_uint64),
        ("decode_calls", C.c_uint64), ("decode_tokens", C.c_uint64),
        ("reclaims", C.c_uint64), ("migrated_blocks", C.c_uint64), ("migrated_bytes", C.c_uint64),
        ("plans_built", C.c_uint64), ("kernel_launches", C.c_uint64),
        ("last_cuda_error", C.c_int32), ("device_status", C.c_int32),
    ]

    def as_dict(self):
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


class SlicePreemptStats(C.Structure):
    _fields_ = [
        ("preempt_oom", C.c_uint64), ("preempt_reclaim", C.c_uint64), ("now", C.c_uint64),
        ("window", C.c_uint64), ("cap_until", C.c_uint64), ("cap_level", C.c_uint64),
    ]

    def as_dict(self):
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


_lib = None


def lib() -> C.CDLL:
    """Loads the CUDA library; raises when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with paper_2609_27040_b200/build.py "
                               "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        u32, u64, i32, vp = C.c_uint32, C.c_uint64, C.c_int32, C.c_void_p
        L.slice_create.argtypes = [C.POINTER(SliceConfig), C.POINTER(vp)]
        L.slice_destroy.argtypes = [vp]
        L.slice_alloc_blocks.argtypes = [vp, i32, u32, i32, vp]
        L.slice_set_seq_len.argtypes = [vp, i32, u32]
        L.slice_free_seq.argtypes = [vp, i32]
        L.slice_get_block_table.argtypes = [vp, i32, vp, u32, vp, vp]
        L.slice_get_free_stack.argtypes = [vp, i32, vp, u32, vp]
        L.prefetch_layer.argtypes = [vp, u32, vp, u32, vp]
        L.paged_decode.argtypes = [vp, u32, vp, u32, vp, u32, C.c_float, vp, vp, vp]
        L.paged_decode_noalloc.argtypes = [vp, u32, vp, u32, vp, u32, C.c_float, vp, vp, vp]
        L.slice_reclaim.argtypes = [vp, u32, vp, vp]
        L.slice_lend.argtypes = [vp, u32]
        L.slice_reclaim_preempt.argtypes = [vp, u32, u32, vp, u32, vp, vp, vp]
        L.slice_preempt_seq.argtypes = [vp, C.c_int32, C.c_int32]
        L.slice_set_preempt_window.argtypes = [vp, C.c_uint64]
        L.slice_set_time.argtypes = [vp, C.c_uint64]
        L.slice_preempt_stats.argtypes = [vp, vp]
        L.slice_set_peer_used.argtypes = [vp, u32]
        L.slice_schedule_gll.argtypes = [vp, u32, vp]
        L.slice_append_kv.argtypes = [vp, u32, vp, u32, vp, vp, vp]
        L.slice_writeback_layer.argtypes = [vp, u32, vp, u32, vp]
        L.slice_decode_step.argtypes = [vp, vp, u32, vp, u32, C.c_float, vp, i32, i32, vp, vp]
        L.slice_step_begin.argtypes = [vp, vp, u32, vp, u32, C.c_float, vp, i32, vp]
        L.slice_step_submit_q.argtypes = [vp, u32, vp]
        L.slice_step_wait_out.argtypes = [vp, u32, vp]
        L.slice_step_flags.argtypes = [vp, vp, vp, vp]
        L.slice_step_relay.argtypes = [vp, vp]
        L.slice_stats.argtypes = [vp, C.POINTER(SliceStats)]
        L.slice_get_resolved.argtypes = [vp, vp, u32, vp, u32, vp]
        L.slice_layer_times.argtypes = [vp, vp, u32]
        L.slice_cta_trace.argtypes = [vp, i32, vp, u64, vp, vp]
        L.slice_copy_blocks.argtypes = [vp, vp, vp, vp, u32, u64, u32, u32, vp]
        L.slice_copy_blocks_series.argtypes = [vp, u32, u64, vp, vp, u64, u32, u64, i32, u32, u32, vp]
        L.slice_strerror.argtypes = [C.c_int]
        L.slice_strerror.restype = C.c_char_p
        _lib = L
    return _lib


def slice_strerror(code: int) -> str:
    return lib().slice_strerror(code).decode()


class SliceError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {slice_strerror(code)} ({code})")
        self.code = code


def _ptr(x) -> Optional[int]:
    """Address of a numpy array, a torch tensor, an int or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        assert x.flags["C_CONTIGUOUS"]
        return x.ctypes.data
    return x.data_ptr()  # torch tensor


def _stream(s) -> Optional[int]:
    if s is None or isinstance(s, int):
        return s
    return s.cuda_stream  # torch.cuda.Stream


def _seqs(seqs) -> np.ndarray:
    return np.ascontiguousarray(seqs, np.int32)


def kv_block_swizzle(x):
    """Converts KV rows between canonical order and the block format's storage order (and back: the
    permutation is its own inverse). `x` is a numpy array or torch tensor of 16-bit elements whose
    last three dimensions are [16 token rows][num_kv_heads][128]; within every 128 bytes of token
    row r, the 16-byte unit u moves to unit u ^ (r & 7). Returns a new array."""
    shape = tuple(x.shape)
    if len(shape) < 3 or shape[-3] != 16 or shape[-1] != 128:
        raise ValueError(f"expected [..., 16, num_kv_heads, 128], got {shape}")
    v = x.reshape(shape[:-3] + (16, shape[-2] * 2, 8, 8))
    out = v.copy() if isinstance(v, np.ndarray) else v.clone()
    for k in range(1, 8):
        perm = [u ^ k for u in range(8)]
        out[..., k::8, :, :, :] = v[..., k::8, :, perm, :]
    return out.reshape(shape)


ALL_LAYERS = 0xFFFFFFFF


class Slice:
    """Owner of one ``slice_t`` handle. Methods are named after the C entry points and return the
    status code (plus outputs); ``check=True`` turns a non-zero status into SliceError."""

    def __init__(self, num_layers: int, num_kv_heads: int, local_blocks: int, lent_blocks: int,
                 staging_blocks_per_slot: int, local=None, lent=None, staging=None,
                 lent_blocks_physical: Optional[int] = None, ring_slots: int = 2, max_seqs: int = 256,
                 max_blocks_per_seq: int = 512, head_dim: int = 128, block_tokens: int = 16,
                 lent_kind: int = 0, flags: int = 0, local_free_order=None, lent_free_order=None,
                 decode_ctas: int = 0, copy_ctas: int = 0, copy_kind: int = 0, pipeline_mode: int = 0,
                 static_split: int = 0, claim_blocks: int = 0, steal_floor: int = 0, prefetch_priority: int = 0,
                 slab_blocks: int = 0, layer_group: int = 0, layout: int = 0, split_layer: int = 0, swap_out: int = 0,
                 local_layer_stride: int = 0, local_block_stride: int = 0,
                 lent_layer_stride: int = 0, lent_block_stride: int = 0):
        cfg = SliceConfig()
        cfg.num_layers, cfg.num_kv_heads, cfg.head_dim, cfg.block_tokens, cfg.dtype = \
            num_layers, num_kv_heads, head_dim, block_tokens, 0
        cfg.local_blocks, cfg.lent_blocks = local_blocks, lent_blocks
        cfg.lent_blocks_physical = lent_blocks if lent_blocks_physical is None else lent_blocks_physical
        cfg.ring_slots, cfg.staging_blocks_per_slot = ring_slots, staging_blocks_per_slot
        cfg.max_seqs, cfg.max_blocks_per_seq = max_seqs, max_blocks_per_seq
        cfg.lent_kind, cfg.flags = lent_kind, flags
        cfg.local_base, cfg.lent_base, cfg.staging_base = _ptr(local), _ptr(lent), _ptr(staging)
        cfg.local_layer_stride, cfg.local_block_stride = local_layer_stride, local_block_stride
        cfg.lent_layer_stride, cfg.lent_block_stride = lent_layer_stride, lent_block_stride
        self._lo = None if local_free_order is None else np.ascontiguousarray(local_free_order, np.uint32)
        self._ro = None if lent_free_order is None else np.ascontiguousarray(lent_free_order, np.uint32)
        cfg.local_free_order, cfg.lent_free_order = _ptr(self._lo), _ptr(self._ro)
        cfg.decode_ctas, cfg.copy_ctas, cfg.copy_kind = decode_ctas, copy_ctas, copy_kind
        cfg.pipeline_mode, cfg.static_split = pipeline_mode, static_split
        cfg.claim_blocks, cfg.steal_floor, cfg.prefetch_priority = claim_blocks, steal_floor, prefetch_priority
        cfg.slab_blocks, cfg.layer_group, cfg.layout = slab_blocks, layer_group, layout
        cfg.split_layer, cfg.swap_out = split_layer, swap_out
        self.cfg = cfg
        self._keep = (local, lent, staging)       # arenas must outlive the slice
        h = C.c_void_p()
        rc = lib().slice_create(C.byref(cfg), C.byref(h))
        if rc != OK:
            raise SliceError(rc, "slice_create")
        self._h = h
        self.max_blocks_per_seq = max_blocks_per_seq
        self.num_layers = num_layers

    # -- lifetime ---------------------------------------------------------------------------
    def slice_destroy(self):
        if self._h:
            lib().slice_destroy(self._h)
            self._h = None

    close = slice_destroy

    def __del__(self):
        try:
            self.slice_destroy()
        except Exception:
            pass

    # -- allocator --------------------------------------------------------------------------
    def slice_alloc_blocks(self, seq: int, n: int, tier_hint: int = TIER_AUTO):
        out = np.zeros(max(n, 1), np.int32)
        rc = lib().slice_alloc_blocks(self._h, seq, n, tier_hint, _ptr(out))
        return rc, out[:n]

    def slice_set_seq_len(self, seq: int, length: int) -> int:
        return lib().slice_set_seq_len(self._h, seq, length)

    def slice_free_seq(self, seq: int) -> int:
        return lib().slice_free_seq(self._h, seq)

    def slice_get_block_table(self, seq: int):
        n, ln = C.c_uint32(0), C.c_uint32(0)
        rc = lib().slice_get_block_table(self._h, seq, None, 0, C.byref(n), C.byref(ln))
        if rc != OK:
            return rc, None, 0
        out = np.zeros(max(n.value, 1), np.int32)
        rc = lib().slice_get_block_table(self._h, seq, _ptr(out), n.value, C.byref(n), C.byref(ln))
        return rc, out[:n.value], ln.value

    def slice_get_free_stack(self, tier: int) -> np.ndarray:
        n = C.c_uint32(0)
        lib().slice_get_free_stack(self._h, tier, None, 0, C.byref(n))
        out = np.zeros(max(n.value, 1), np.int32)
        lib().slice_get_free_stack(self._h, tier, _ptr(out), n.value, C.byref(n))
        return out[:n.value]

    # -- data path --------------------------------------------------------------------------
    def prefetch_layer(self, layer: int, seqs, side_stream=None) -> int:
        sq = _seqs(seqs)
        return lib().prefetch_layer(self._h, layer, _ptr(sq), len(sq), _stream(side_stream))

    def paged_decode(self, layer: int, seqs, q, num_q_heads: int, sm_scale: float, out, lse=None,
                     stream=None) -> int:
        sq = _seqs(seqs)
        return lib().paged_decode(self._h, layer, _ptr(sq), len(sq), _ptr(q), num_q_heads, sm_scale,
                                  _ptr(out), _ptr(lse), _stream(stream))

    def paged_decode_noalloc(self, layer: int, seqs, q, num_q_heads: int, sm_scale: float, out, lse=None,
                             stream=None) -> int:
        """paged_decode for callers that must not allocate device memory: same arguments and result,
        scratch in the library's static 8 MiB device array (see include/emaslice.h for the limit, the
        one-time set-up on the first call per device, and the rule against overlapping calls)."""
        sq = _seqs(seqs)
        return lib().paged_decode_noalloc(self._h, layer, _ptr(sq), len(sq), _ptr(q), num_q_heads, sm_scale,
                                          _ptr(out), _ptr(lse), _stream(stream))

    def slice_reclaim(self, take_blocks: int = TAKE_ALL, stream=None):
        mig = C.c_uint64(0)
        rc = lib().slice_reclaim(self._h, take_blocks, C.byref(mig), _stream(stream))
        return rc, mig.value

    def slice_lend(self, n_blocks: int) -> int:
        return lib().slice_lend(self._h, n_blocks)

    def slice_reclaim_preempt(self, take_blocks: int = TAKE_ALL, slab_blocks: int = 10, stream=None,
                              max_victims: int = None):
        """Returns (rc, preempted sequence ids in eviction order, migrated blocks)."""
        cap = int(self.cfg.max_seqs) if max_victims is None else max_victims
        victims = np.zeros(max(cap, 1), np.int32)
        n, mig = C.c_uint32(0), C.c_uint64(0)
        rc = lib().slice_reclaim_preempt(self._h, take_blocks, slab_blocks, _ptr(victims), cap, C.byref(n),
                                         C.byref(mig), _stream(stream))
        return rc, victims[:n.value].tolist(), mig.value

    def slice_preempt_seq(self, seq: int, cause: int) -> int:
        return lib().slice_preempt_seq(self._h, seq, cause)

    def slice_set_preempt_window(self, window: int) -> int:
        return lib().slice_set_preempt_window(self._h, window)

    def slice_set_time(self, now: int) -> int:
        return lib().slice_set_time(self._h, now)

    def slice_set_peer_used(self, peer_blocks: int) -> int:
        return lib().slice_set_peer_used(self._h, peer_blocks)

    def slice_preempt_stats(self) -> dict:
        st = SlicePreemptStats()
        rc = lib().slice_preempt_stats(self._h, C.byref(st))
        if rc != OK:
            raise SliceError(rc, "slice_preempt_stats")
        return st.as_dict()

    def slice_append_kv(self, layer: int, seqs, k_new, v_new, stream=None) -> int:
        sq = _seqs(seqs)
        return lib().slice_append_kv(self._h, layer, _ptr(sq), len(sq), _ptr(k_new), _ptr(v_new),
                                     _stream(stream))

    def slice_writeback_layer(self, layer: int, seqs, stream=None) -> int:
        sq = _seqs(seqs)
        return lib().slice_writeback_layer(self._h, layer, _ptr(sq), len(sq), _stream(stream))

    def slice_decode_step(self, seqs, q, num_q_heads: int, sm_scale: float, out, io_on_host: bool = False,
                          wrap_prefetch: bool = True, stream=None, side_stream=None) -> int:
        sq = seqs if isinstance(seqs, np.ndarray) and seqs.dtype == np.int32 else _seqs(seqs)
        return lib().slice_decode_step(self._h, _ptr(sq), len(sq), _ptr(q), num_q_heads, sm_scale, _ptr(out),
                                       int(io_on_host), int(wrap_prefetch), _stream(stream),
                                       _stream(side_stream))

    def slice_step_begin(self, seqs, q, num_q_heads: int, sm_scale: float, out, wrap_prefetch: bool = True,
                         stream=None) -> int:
        sq = seqs if isinstance(seqs, np.ndarray) and seqs.dtype == np.int32 else _seqs(seqs)
        return lib().slice_step_begin(self._h, _ptr(sq), len(sq), _ptr(q), num_q_heads, sm_scale, _ptr(out),
                                      int(wrap_prefetch), _stream(stream))

    def slice_step_submit_q(self, layer: int, caller_stream) -> int:
        return lib().slice_step_submit_q(self._h, layer, _stream(caller_stream))

    def slice_step_wait_out(self, layer: int, caller_stream) -> int:
        return lib().slice_step_wait_out(self._h, layer, _stream(caller_stream))

    def slice_step_relay(self, caller_stream) -> int:
        return lib().slice_step_relay(self._h, _stream(caller_stream))

    def slice_step_flags(self):
        """(rc, device address of q_ready[], device address of out_ready[], epoch of the pass begun last)."""
        qr, orr, ep = C.c_void_p(), C.c_void_p(), C.c_uint32(0)
        rc = lib().slice_step_flags(self._h, C.byref(qr), C.byref(orr), C.byref(ep))
        return rc, qr.value, orr.value, ep.value

    # -- introspection ----------------------------------------------------------------------
    def slice_stats(self) -> dict:
        st = SliceStats()
        rc = lib().slice_stats(self._h, C.byref(st))
        if rc != OK:
            raise SliceError(rc, "slice_stats")
        return st.as_dict()

    def slice_get_resolved(self, seqs):
        sq = _seqs(seqs)
        out = np.full((len(sq), self.max_blocks_per_seq), np.iinfo(np.int32).min, np.int32)
        k = C.c_uint32(0)
        rc = lib().slice_get_resolved(self._h, _ptr(sq), len(sq), _ptr(out), out.size, C.byref(k))
        return rc, out, k.value

    def slice_layer_times(self) -> np.ndarray:
        out = np.zeros((self.num_layers, 5), np.float32)
        rc = lib().slice_layer_times(self._h, _ptr(out), self.num_layers)
        if rc != OK:
            raise SliceError(rc, "slice_layer_times")
        return out


def _cta_trace(self, which: int) -> np.ndarray:
    per, words = C.c_uint32(0), C.c_uint32(0)
    rc = lib().slice_cta_trace(self._h, which, None, 0, C.byref(per), C.byref(words))
    if rc != OK:
        raise SliceError(rc, "slice_cta_trace")
    out = np.zeros((self.num_layers, per.value, words.value), np.uint64)
    rc = lib().slice_cta_trace(self._h, which, _ptr(out), out.size, C.byref(per), C.byref(words))
    if rc != OK:
        raise SliceError(rc, "slice_cta_trace")
    return out


Slice.slice_cta_trace = _cta_trace


def slice_copy_blocks(dst, dst_idx, src, src_idx, n: int, block_bytes: int, kind: int = 0, ctas: int = 0,
                      stream=None) -> int:
    return lib().slice_copy_blocks(_ptr(dst), _ptr(dst_idx), _ptr(src), _ptr(src_idx), n, block_bytes, kind,
                                   ctas, _stream(stream))


def slice_copy_blocks_series(ring, ring_slots: int, slot_bytes: int, arena, idx, n_total: int, per_launch: int,
                             block_bytes: int, scatter: bool = False, kind: int = 0, ctas: int = 0, stream=None) -> int:
    return lib().slice_copy_blocks_series(_ptr(ring), ring_slots, slot_bytes, _ptr(arena), _ptr(idx), n_total, per_launch,
                                          block_bytes, int(scatter), kind, ctas, _stream(stream))


def slice_schedule_gll(slices) -> int:
    """Index of the slice a new request goes to (Greedy-Least-Loaded over Slice objects)."""
    arr = (C.c_void_p * len(slices))(*[sl._h for sl in slices])
    out = C.c_uint32(0)
    rc = lib().slice_schedule_gll(arr, len(slices), C.byref(out))
    if rc != OK:
        raise SliceError(rc, "slice_schedule_gll")
    return int(out.value)
