"""ctypes front end of the CPU oracle (``ema_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the benchmark's
CPU-baseline leg. The product package never imports this module and shares no code with it.

Arrays are numpy; bf16 tensors travel as ``uint16`` bit patterns. Every function cites, in the
C++ source, the passage of the paper it follows.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ema_oracle.cpp")
_LIB = os.path.join(_HERE, "libema_oracle.so")

OK, E_INVAL, E_NOSPC, E_STAGING, E_STATE, E_CAPPED = 0, -1, -2, -3, -7, -9
PREEMPT_OOM, PREEMPT_RECLAIM = 1, 2
AUTO, LOCAL, LENT = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2, OpenMP). Returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        u32, u64, i32, vp = C.c_uint32, C.c_uint64, C.c_int32, C.c_void_p
        L.oracle_create.restype = vp
        L.oracle_create.argtypes = [u32, u32, u64, u32, u32, u32, u32, u32, u32, u32, vp, vp]
        L.oracle_destroy.argtypes = [vp]
        L.oracle_destroy.restype = None
        L.oracle_alloc_blocks.argtypes = [vp, i32, u32, i32, vp]
        L.oracle_set_seq_len.argtypes = [vp, i32, u32]
        L.oracle_free_seq.argtypes = [vp, i32]
        L.oracle_get_block_table.argtypes = [vp, i32, vp, u32, vp, vp]
        L.oracle_get_free_stack.argtypes = [vp, i32, vp, u32, vp]
        L.oracle_lent_capacity.argtypes = [vp]
        L.oracle_lent_capacity.restype = u32
        L.oracle_num_seqs.argtypes = [vp]
        L.oracle_num_seqs.restype = u32
        L.oracle_gather.argtypes = [vp, u32, vp, u32, vp, vp, vp, vp]
        L.oracle_scatter.argtypes = [vp, u32, vp, u32, vp, vp]
        L.oracle_paged_attention.argtypes = [vp, vp, vp, vp, u32, vp, u32, u32, u32, u32, u32,
                                             C.c_double, vp, vp]
        L.oracle_dense_attention.argtypes = [vp, vp, vp, u32, u32, u32, u32, C.c_double, vp, vp, vp]
        L.oracle_to_bf16.argtypes = [vp, vp, u64]
        L.oracle_to_bf16.restype = None
        L.oracle_reclaim.argtypes = [vp, u32, vp, vp, vp]
        L.oracle_lend.argtypes = [vp, u32]
        L.oracle_set_preempt_window.argtypes = [vp, u64]
        L.oracle_set_time.argtypes = [vp, u64]
        L.oracle_preempt_seq.argtypes = [vp, i32, i32]
        L.oracle_reclaim_preempt.argtypes = [vp, u32, u32, vp, vp, vp, u32, vp, vp]
        L.oracle_preempt_state.argtypes = [vp, vp]
        L.oracle_preempt_state.restype = None
        L.oracle_append_kv.argtypes = [vp, u32, vp, u32, vp, vp, u32, u32, vp, vp, vp]
        L.oracle_num_threads.restype = C.c_int
        L.oracle_set_slab_blocks.argtypes = [vp, u32]
        L.oracle_layout_offset.argtypes = [u32, u32, u32, u32, u32, u64, u32, u32]
        L.oracle_layout_offset.restype = u64
        L.oracle_swap_pieces.argtypes = [u32, u32, u32, u32, u32, u64, u32, vp, u32, vp, u32]
        L.oracle_swap_pieces.restype = u32
    return _lib


def _ptr(a: Optional[np.ndarray]):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.c_void_p)


def num_threads() -> int:
    return int(lib().oracle_num_threads())


class OracleSlice:
    """Integer state machine of one slice plus the byte-moving steps on host arenas."""

    def __init__(self, num_layers: int, block_tokens: int, block_bytes: int, local_blocks: int,
                 lent_blocks: int, lent_physical: Optional[int] = None, ring_slots: int = 2,
                 staging_blocks_per_slot: int = 0, max_seqs: int = 1024,
                 max_blocks_per_seq: int = 1024,
                 local_free_order: Optional[np.ndarray] = None,
                 lent_free_order: Optional[np.ndarray] = None):
        self.num_layers = num_layers
        self.block_tokens = block_tokens
        self.block_bytes = block_bytes
        self.local_blocks = local_blocks
        self.lent_physical = lent_blocks if lent_physical is None else lent_physical
        self.ring_slots = ring_slots
        self.staging_cap = staging_blocks_per_slot
        self.max_seqs = max_seqs
        self.max_blocks_per_seq = max_blocks_per_seq
        lo = None if local_free_order is None else np.ascontiguousarray(local_free_order, np.uint32)
        ro = None if lent_free_order is None else np.ascontiguousarray(lent_free_order, np.uint32)
        self._h = lib().oracle_create(num_layers, block_tokens, block_bytes, local_blocks,
                                      lent_blocks, self.lent_physical, ring_slots,
                                      staging_blocks_per_slot, max_seqs, max_blocks_per_seq,
                                      _ptr(lo), _ptr(ro))
        if not self._h:
            raise ValueError("oracle_create: bad configuration")

    def close(self):
        if self._h:
            lib().oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- allocator --------------------------------------------------------------------------
    def alloc_blocks(self, seq: int, n: int, hint: int = AUTO):
        out = np.zeros(max(n, 1), np.int32)
        rc = lib().oracle_alloc_blocks(self._h, seq, n, hint, _ptr(out))
        return rc, out[:n]

    def set_seq_len(self, seq: int, length: int) -> int:
        return lib().oracle_set_seq_len(self._h, seq, length)

    def set_slab_blocks(self, slab_blocks: int) -> int:
        """Slab allocator of Section 4.2.1 (0 = off). Before the first allocation."""
        return lib().oracle_set_slab_blocks(self._h, slab_blocks)

    def free_seq(self, seq: int) -> int:
        return lib().oracle_free_seq(self._h, seq)

    def block_table(self, seq: int):
        n, ln = C.c_uint32(0), C.c_uint32(0)
        rc = lib().oracle_get_block_table(self._h, seq, None, 0, C.byref(n), C.byref(ln))
        if rc != OK:
            return rc, None, 0
        out = np.zeros(max(n.value, 1), np.int32)
        rc = lib().oracle_get_block_table(self._h, seq, _ptr(out), n.value, C.byref(n), C.byref(ln))
        return rc, out[:n.value], ln.value

    def free_stack(self, which: int) -> np.ndarray:
        n = C.c_uint32(0)
        lib().oracle_get_free_stack(self._h, which, None, 0, C.byref(n))
        out = np.zeros(max(n.value, 1), np.int32)
        lib().oracle_get_free_stack(self._h, which, _ptr(out), n.value, C.byref(n))
        return out[:n.value]

    @property
    def lent_capacity(self) -> int:
        return int(lib().oracle_lent_capacity(self._h))

    @property
    def num_seqs(self) -> int:
        return int(lib().oracle_num_seqs(self._h))

    # -- data movement ----------------------------------------------------------------------
    def gather(self, layer: int, seqs: Sequence[int], lent_arena: Optional[np.ndarray],
               staging: Optional[np.ndarray]):
        """Returns (rc, resolved [nseq][max_blocks_per_seq] int32, k)."""
        sq = np.ascontiguousarray(seqs, np.int32)
        resolved = np.full((len(sq), self.max_blocks_per_seq), np.iinfo(np.int32).min, np.int32)
        k = C.c_uint32(0)
        rc = lib().oracle_gather(self._h, layer, _ptr(sq), len(sq), _ptr(lent_arena), _ptr(staging),
                                 _ptr(resolved), C.byref(k))
        return rc, resolved, k.value

    def scatter(self, layer: int, seqs: Sequence[int], staging: np.ndarray, lent_arena: np.ndarray) -> int:
        sq = np.ascontiguousarray(seqs, np.int32)
        return lib().oracle_scatter(self._h, layer, _ptr(sq), len(sq), _ptr(staging), _ptr(lent_arena))

    def reclaim(self, take: int, local_arena: Optional[np.ndarray], lent_arena: Optional[np.ndarray]):
        mig = C.c_uint64(0)
        rc = lib().oracle_reclaim(self._h, min(take, 0xFFFFFFFF), _ptr(local_arena), _ptr(lent_arena),
                                  C.byref(mig))
        return rc, mig.value

    def lend(self, n: int) -> int:
        return lib().oracle_lend(self._h, n)

    # -- preemption ---------------------------------------------------------------------------
    def set_preempt_window(self, window: int) -> int:
        return lib().oracle_set_preempt_window(self._h, window)

    def set_time(self, now: int) -> int:
        return lib().oracle_set_time(self._h, now)

    def preempt_seq(self, seq: int, cause: int) -> int:
        return lib().oracle_preempt_seq(self._h, seq, cause)

    def reclaim_preempt(self, take: int, slab_blocks: int, local_arena: Optional[np.ndarray],
                        lent_arena: Optional[np.ndarray], max_victims: Optional[int] = None):
        """Returns (rc, evicted sequence ids in eviction order, migrated blocks)."""
        cap = self.max_seqs if max_victims is None else max_victims
        victims = np.zeros(max(cap, 1), np.int32)
        n, mig = C.c_uint32(0), C.c_uint64(0)
        rc = lib().oracle_reclaim_preempt(self._h, min(take, 0xFFFFFFFF), slab_blocks, _ptr(local_arena),
                                          _ptr(lent_arena), _ptr(victims), cap, C.byref(n), C.byref(mig))
        return rc, victims[:n.value].tolist(), mig.value

    def preempt_state(self) -> dict:
        out = np.zeros(6, np.uint64)
        lib().oracle_preempt_state(self._h, _ptr(out))
        keys = ("preempt_oom", "preempt_reclaim", "now", "window", "cap_until", "cap_level")
        return {k: int(v) for k, v in zip(keys, out)}

    def append_kv(self, layer: int, seqs: Sequence[int], k_new: np.ndarray, v_new: np.ndarray,
                  num_kv_heads: int, head_dim: int, local_arena: np.ndarray, lent_arena: np.ndarray,
                  staging_slot: Optional[np.ndarray]) -> int:
        sq = np.ascontiguousarray(seqs, np.int32)
        return lib().oracle_append_kv(self._h, layer, _ptr(sq), len(sq), _ptr(k_new), _ptr(v_new),
                                      num_kv_heads, head_dim, _ptr(local_arena), _ptr(lent_arena),
                                      _ptr(staging_slot))


def paged_attention(q: np.ndarray, local_layer: np.ndarray, staging_slot: Optional[np.ndarray],
                    resolved: np.ndarray, lens: np.ndarray, num_q_heads: int, num_kv_heads: int,
                    head_dim: int, block_tokens: int, sm_scale: float, want_lse: bool = True):
    """fp64 paged decode attention. q: uint16 [nseq][Hq][D]; arenas: uint16, one layer."""
    nseq = q.shape[0]
    resolved = np.ascontiguousarray(resolved, np.int32)
    lens = np.ascontiguousarray(lens, np.uint32)
    out = np.zeros((nseq, num_q_heads, head_dim), np.float64)
    lse = np.zeros((nseq, num_q_heads), np.float64) if want_lse else None
    rc = lib().oracle_paged_attention(_ptr(q), _ptr(local_layer), _ptr(staging_slot), _ptr(resolved),
                                      resolved.shape[1], _ptr(lens), nseq, num_q_heads, num_kv_heads,
                                      head_dim, block_tokens, float(sm_scale), _ptr(out), _ptr(lse))
    return rc, out, lse


def dense_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, num_q_heads: int, num_kv_heads: int,
                    head_dim: int, sm_scale: float, want_probs: bool = False):
    """Brute force for one sequence. q: uint16 [Hq][D]; K, V: uint16 [n][Hkv][D]."""
    n = K.shape[0]
    out = np.zeros((num_q_heads, head_dim), np.float64)
    lse = np.zeros((num_q_heads,), np.float64)
    probs = np.zeros((num_q_heads, n), np.float64) if want_probs else None
    rc = lib().oracle_dense_attention(_ptr(q), _ptr(K), _ptr(V), n, num_q_heads, num_kv_heads,
                                      head_dim, float(sm_scale), _ptr(out), _ptr(lse), _ptr(probs))
    return rc, out, lse, probs


def to_bf16(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, np.float64)
    y = np.zeros(x.shape, np.uint16)
    lib().oracle_to_bf16(_ptr(x), _ptr(y), x.size)
    return y


# -- scheduling across slices (O-schedule) --------------------------------------------------------
def gll_choose(own_blocks: Sequence[int], peer_blocks: Sequence[int], capacity_blocks: Sequence[int]) -> int:
    """Section 5.2 / Appendix C, Greedy-Least-Loaded: a request goes to the incident slice k with the
    smallest util_{k,i} + util_{k,j}, each utilisation being blocks held over the slice's capacity.
    Exact rational arithmetic; among equals the first slice. Returns -1 for an empty list."""
    from fractions import Fraction
    best, best_u = -1, None
    for k, (a, b, c) in enumerate(zip(own_blocks, peer_blocks, capacity_blocks)):
        if c <= 0:
            raise ValueError("slice without capacity")
        u = Fraction(int(a), int(c)) + Fraction(int(b), int(c))
        if best_u is None or u < best_u:
            best, best_u = k, u
    return best


# -- memory layouts (O-slab) ------------------------------------------------------------------------
LAYER_MAJOR, SLAB_MAJOR, LAYER_GROUP_MAJOR = 0, 1, 2


def layout_offset(layout: int, num_layers: int, n_blocks: int, slab_blocks: int, layer_group: int,
                  block_bytes: int, layer: int, block_id: int) -> int:
    """Byte offset of a block in an arena laid out as Section 4.2.1 / 4.2.2 / 4.2.3 describes."""
    return int(lib().oracle_layout_offset(layout, num_layers, n_blocks, slab_blocks, layer_group, block_bytes,
                                          layer, block_id))


def swap_pieces(layout: int, num_layers: int, n_blocks: int, slab_blocks: int, layer_group: int,
                block_bytes: int, group: int, slabs: Sequence[int]) -> list:
    """Lengths in bytes of the contiguous pieces one swap of `group` moves for the owner of `slabs`."""
    sl = np.ascontiguousarray(slabs, np.uint32)
    n = lib().oracle_swap_pieces(layout, num_layers, n_blocks, slab_blocks, layer_group, block_bytes, group,
                                 _ptr(sl), len(sl), None, 0)
    out = np.zeros(max(n, 1), np.uint64)
    lib().oracle_swap_pieces(layout, num_layers, n_blocks, slab_blocks, layer_group, block_bytes, group,
                             _ptr(sl), len(sl), _ptr(out), n)
    return [int(x) for x in out[:n]]


def group_layers(layer_group: int, group: int) -> range:
    """Section 4.2.2: a layer group is a set of logically consecutive layers; group g of size k holds
    layers g*k .. g*k + k - 1, and is handled like one big layer."""
    return range(group * layer_group, (group + 1) * layer_group)
