"""Host-side scenario builder shared by the oracle pins and the GPU parity tests.

It replays a seeded placement on the oracle's integer state machine, fills numpy arenas with
bf16 bit patterns, and keeps the dense logical K/V of every (sequence, layer) for brute force.
Nothing here computes gather, attention or migration: those come from ``oracle`` (CPU) or from the
CUDA library, and the tests compare the two.
"""
from __future__ import annotations

import numpy as np

import oracle
from paper_2609_27040_b200 import synth


class Scenario:
    def __init__(self, wl: synth.Workload, seed: int, poison: bool = False, slack: int = 16,
                 num_layers: int | None = None, lent_extra_physical: int = 0,
                 lengths: np.ndarray | None = None, permute: bool = True,
                 max_blocks_per_seq: int | None = None, slab_blocks: int = 0):
        self.wl = wl
        self.seed = seed
        self.L = wl.num_layers if num_layers is None else num_layers
        self.T, self.Hkv, self.Hq, self.D = wl.block_tokens, wl.num_kv_heads, wl.num_q_heads, wl.head_dim
        self.slab = slab_blocks
        self.pl = synth.make_placement(wl, seed, slack_blocks=slack, permute=permute and not slab_blocks, lengths=lengths)
        pl = self.pl
        if slab_blocks:          # slab allocator: whole slabs, ids in the order the slab rule gives (no seeded order)
            pl.local_blocks = -(-pl.local_blocks // slab_blocks) * slab_blocks
            pl.lent_blocks = -(-(pl.lent_blocks + lent_extra_physical) // slab_blocks) * slab_blocks - lent_extra_physical
        self.nseq = len(pl.lengths)
        self.lent_phys = pl.lent_blocks + lent_extra_physical
        self.staging_cap = max(pl.staging_blocks, 1)
        self.max_blocks = max_blocks_per_seq or max(int(max(len(h) for h in pl.hints)) + 2, 4)
        rng = np.random.default_rng(seed + 1000)
        if lent_extra_physical and pl.lent_free_order is not None:
            # the free order must be a permutation of the whole physical arena
            self.lent_order = synth.free_order(rng, self.lent_phys)
        else:
            self.lent_order = pl.lent_free_order
        self.local_order = pl.local_free_order
        self.orc = oracle.OracleSlice(self.L, self.T, wl.block_bytes, pl.local_blocks, pl.lent_blocks,
                                      self.lent_phys, wl.ring_slots, self.staging_cap,
                                      max_seqs=max(self.nseq, 1) + 4, max_blocks_per_seq=self.max_blocks,
                                      local_free_order=self.local_order, lent_free_order=self.lent_order)
        if slab_blocks:
            assert self.orc.set_slab_blocks(slab_blocks) == oracle.OK
        self.seq_ids = list(pl.seq_ids)
        # one allocation call per block, in logical order, with the drawn tier hint
        for i, hints in zip(self.seq_ids, pl.hints):
            for hnt in hints:
                rc, _ = self.orc.alloc_blocks(i, 1, int(hnt))
                assert rc == oracle.OK
            assert self.orc.set_seq_len(i, int(pl.lengths[i])) == oracle.OK
        shape_blk = (2, self.T, self.Hkv, self.D)
        if poison:
            self.local = np.full((self.L, pl.local_blocks) + shape_blk, synth.BF16_NAN, np.uint16)
            self.lent = np.full((self.L, self.lent_phys) + shape_blk, synth.BF16_NAN, np.uint16)
            self.staging = np.full((wl.ring_slots, self.staging_cap) + shape_blk, synth.BF16_NAN, np.uint16)
        else:
            fill = np.random.default_rng(seed + 2000)      # background bytes: a stream of their own
            self.local = synth.normal_bf16_bits(fill, (self.L, pl.local_blocks) + shape_blk)
            self.lent = synth.normal_bf16_bits(fill, (self.L, self.lent_phys) + shape_blk)
            self.staging = synth.normal_bf16_bits(fill, (wl.ring_slots, self.staging_cap) + shape_blk)
        # logical data: dense K/V per (seq, layer), written through the oracle's tables
        self.dense = {}
        for i in self.seq_ids:
            n = int(pl.lengths[i])
            rc, table, _ = self.orc.block_table(i)
            assert rc == oracle.OK
            for l in range(self.L):
                K = synth.normal_bf16_bits(rng, (n, self.Hkv, self.D))
                V = synth.normal_bf16_bits(rng, (n, self.Hkv, self.D))
                self.dense[(i, l)] = (K, V)
                self.write_logical(i, l, K, V, table)
        self.q = synth.normal_bf16_bits(rng, (self.L, self.nseq, self.Hq, self.D))
        self.sm_scale = 1.0 / np.sqrt(self.D)

    def write_logical(self, seq, layer, K, V, table=None):
        """Store dense K/V rows of one (seq, layer) into the arenas through the block table."""
        if table is None:
            _, table, _ = self.orc.block_table(seq)
        n = K.shape[0]
        for b in range(synth.blocks_for(n, self.T)):
            t0, t1 = b * self.T, min(n, (b + 1) * self.T)
            e = int(table[b])
            blk = self.local[layer, e] if e >= 0 else self.lent[layer, ~e]
            blk[0, : t1 - t0] = K[t0:t1]
            blk[1, : t1 - t0] = V[t0:t1]

    def logical_view(self, seq, layer):
        """Bytes of blocks 0..nb-1 of a sequence, read through its current block table."""
        _, table, _ = self.orc.block_table(seq)
        return np.stack([self.local[layer, e] if e >= 0 else self.lent[layer, ~e] for e in table.tolist()])

    def lengths(self):
        return np.asarray([int(self.pl.lengths[i]) for i in self.seq_ids], np.uint32)


def attention_close(got: np.ndarray, ref: np.ndarray, atol=1e-2, rtol=1e-2):
    """The stated bf16 attention tolerance: |got - ref| <= atol + rtol * |ref| elementwise."""
    err = np.abs(got.astype(np.float64) - ref)
    ok = err <= atol + rtol * np.abs(ref)
    big = np.abs(ref) >= 2.0 ** -6
    max_rel = float((err[big] / np.abs(ref[big])).max()) if big.any() else 0.0
    return bool(ok.all()), float(err.max()), max_rel
