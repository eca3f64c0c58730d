"""Pins of the oracle's paged attention against things other than itself: a dense brute force,
closed forms, invariants, and an fp64 library attention. CPU only."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_27040_b200 import synth
from tests.helpers import Scenario

WL1 = synth.WORKLOADS["single_layer_mha"]
GQA_SMALL = synth.Workload("gqa_small", 2, 32, 8, 5, 40, 300, 0.4)


def _paged(sc: Scenario, layer: int):
    rc, resolved, k = sc.orc.gather(layer, sc.seq_ids, sc.lent, sc.staging)
    assert rc == oracle.OK
    slot = layer % sc.wl.ring_slots
    rc, out, lse = oracle.paged_attention(sc.q[layer], sc.local[layer], sc.staging[slot], resolved,
                                          sc.lengths(), sc.Hq, sc.Hkv, sc.D, sc.T, sc.sm_scale)
    assert rc == oracle.OK
    return out, lse, resolved, k


@pytest.mark.parametrize("wl,seed", [(WL1, 0), (WL1, 1), (GQA_SMALL, 2)])
def test_paged_equals_dense_brute_force(wl, seed):
    """P1: attention over permuted physical blocks (local + staged) == dense contiguous attention."""
    sc = Scenario(wl, seed)
    for layer in range(sc.L):
        out, lse, _, _ = _paged(sc, layer)
        for pos, i in enumerate(sc.seq_ids):
            K, V = sc.dense[(i, layer)]
            rc, ref, ref_lse, _ = oracle.dense_attention(sc.q[layer, pos], K, V, sc.Hq, sc.Hkv, sc.D, sc.sm_scale)
            assert rc == oracle.OK
            assert np.abs(out[pos] - ref).max() <= 1e-12
            assert np.abs(lse[pos] - ref_lse).max() <= 1e-12


def test_softmax_rows_sum_to_one_and_output_is_convex():
    """P2: probabilities sum to 1; each output coordinate lies between min and max of V."""
    sc = Scenario(GQA_SMALL, 3)
    G = sc.Hq // sc.Hkv
    for pos, i in enumerate(sc.seq_ids):
        K, V = sc.dense[(i, 0)]
        _, out, _, probs = oracle.dense_attention(sc.q[0, pos], K, V, sc.Hq, sc.Hkv, sc.D, sc.sm_scale,
                                                  want_probs=True)
        assert np.abs(probs.sum(axis=1) - 1.0).max() <= 1e-12
        assert (probs >= 0).all()
        Vf = synth.bf16_bits_to_f32(V).astype(np.float64)
        for h in range(sc.Hq):
            g = h // G
            assert (out[h] <= Vf[:, g].max(axis=0) + 1e-12).all()
            assert (out[h] >= Vf[:, g].min(axis=0) - 1e-12).all()


def _rand(rng, shape):
    return synth.normal_bf16_bits(rng, shape)


def _f(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def test_closed_forms():
    """P3: special inputs whose answer is known without running attention."""
    rng = np.random.default_rng(7)
    Hq, Hkv, D = 8, 2, 128
    G = Hq // Hkv
    scale = 1 / np.sqrt(D)
    q = _rand(rng, (Hq, D))
    # n = 1: the output is the single V row, exactly
    K, V = _rand(rng, (1, Hkv, D)), _rand(rng, (1, Hkv, D))
    _, out, lse, _ = oracle.dense_attention(q, K, V, Hq, Hkv, D, scale)
    for h in range(Hq):
        assert (out[h] == _f(V)[0, h // G]).all()
        assert abs(lse[h] - scale * (_f(q)[h] @ _f(K)[0, h // G])) <= 1e-12
    # all keys equal: uniform weights, output = mean of V; lse = s + log(n)
    n = 37
    K = np.repeat(_rand(rng, (1, Hkv, D)), n, axis=0)
    V = _rand(rng, (n, Hkv, D))
    _, out, lse, _ = oracle.dense_attention(q, K, V, Hq, Hkv, D, scale)
    for h in range(Hq):
        assert np.abs(out[h] - _f(V)[:, h // G].mean(axis=0)).max() <= 1e-12
        s = scale * (_f(q)[h] @ _f(K)[0, h // G])
        assert abs(lse[h] - (s + np.log(n))) <= 1e-12
    # constant V: output is that constant
    K = _rand(rng, (n, Hkv, D))
    V = np.repeat(_rand(rng, (1, Hkv, D)), n, axis=0)
    _, out, _, _ = oracle.dense_attention(q, K, V, Hq, Hkv, D, scale)
    for h in range(Hq):
        assert np.abs(out[h] - _f(V)[0, h // G]).max() <= 1e-12
    # one dominant key (score gap > 800): output is exactly that key's V row
    K = _rand(rng, (n, Hkv, D))
    V = _rand(rng, (n, Hkv, D))
    qd = np.full((Hq, D), 0x4080, np.uint16)          # 4.0 everywhere
    K[:] = 0
    K[11] = np.uint16(0x4380)                          # 256.0 -> score 4*256*128*scale >> 800
    _, out, _, _ = oracle.dense_attention(qd, K, V, Hq, Hkv, D, scale)
    for h in range(Hq):
        assert (out[h] == _f(V)[11, h // G]).all()


def test_shift_and_permutation_invariance():
    """P3: adding one vector to every key shifts all scores equally; token order is irrelevant."""
    rng = np.random.default_rng(11)
    Hq, Hkv, D, n = 4, 4, 128, 53
    scale = 1 / np.sqrt(D)
    q = _rand(rng, (Hq, D))
    # keys on a coarse grid so that K + u is exactly representable in bf16
    Kf = rng.integers(-8, 9, size=(n, Hkv, D)).astype(np.float32) / 4
    uf = rng.integers(-8, 9, size=(1, Hkv, D)).astype(np.float32) / 4
    to_bits = lambda x: (x.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    K, Ku = to_bits(Kf), to_bits(Kf + uf)
    assert (_f(Ku) == (Kf + uf)).all()
    V = _rand(rng, (n, Hkv, D))
    _, o1, l1, _ = oracle.dense_attention(q, K, V, Hq, Hkv, D, scale)
    _, o2, l2, _ = oracle.dense_attention(q, Ku, V, Hq, Hkv, D, scale)
    assert np.abs(o1 - o2).max() <= 1e-12
    shift = scale * np.einsum("hd,hd->h", _f(q), _f(to_bits(uf))[0])
    assert np.abs((l2 - l1) - shift).max() <= 1e-10
    perm = rng.permutation(n)
    _, o3, l3, _ = oracle.dense_attention(q, K[perm], V[perm], Hq, Hkv, D, scale)
    assert np.abs(o1 - o3).max() <= 1e-12
    assert np.abs(l1 - l3).max() <= 1e-12


@pytest.mark.parametrize("Hq,Hkv", [(8, 8), (32, 8), (64, 8), (12, 4)])
def test_against_fp64_library_attention(Hq, Hkv):
    """P4: grouped-query attention == multi-head attention on KV heads repeated G times, computed
    by torch's scaled_dot_product_attention in fp64 (pins the head mapping and the scale)."""
    rng = np.random.default_rng(5)
    D, n = 128, 211
    scale = 1 / np.sqrt(D)
    q, K, V = _rand(rng, (Hq, D)), _rand(rng, (n, Hkv, D)), _rand(rng, (n, Hkv, D))
    _, out, lse, _ = oracle.dense_attention(q, K, V, Hq, Hkv, D, scale)
    G = Hq // Hkv
    qt = torch.from_numpy(_f(q))[None, :, None, :]                                   # [1,Hq,1,D]
    Kt = torch.from_numpy(_f(K)).permute(1, 0, 2).repeat_interleave(G, dim=0)[None]  # [1,Hq,n,D]
    Vt = torch.from_numpy(_f(V)).permute(1, 0, 2).repeat_interleave(G, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(qt, Kt, Vt, scale=scale)[0, :, 0].numpy()
    assert np.abs(out - ref).max() <= 1e-10
    ref_lse = torch.logsumexp(scale * (qt @ Kt.transpose(-1, -2))[0, :, 0], dim=-1).numpy()
    assert np.abs(lse - ref_lse).max() <= 1e-10


def test_nan_poisoned_tails_do_not_leak():
    """P5: bytes past a sequence's length (block tails, unused blocks, unused staging) are NaN;
    outputs stay finite and equal the clean run's."""
    clean = Scenario(WL1, 4, poison=False)
    dirty = Scenario(WL1, 4, poison=True)
    for layer in range(clean.L):
        o1, l1, _, _ = _paged(clean, layer)
        o2, l2, _, _ = _paged(dirty, layer)
        assert np.isfinite(o2).all() and np.isfinite(l2).all()
        assert (o1 == o2).all() and (l1 == l2).all()


def test_zero_length_is_rejected():
    sc = Scenario(WL1, 0)
    _, resolved, _ = sc.orc.gather(0, sc.seq_ids, sc.lent, sc.staging)
    lens = sc.lengths()
    lens[1] = 0
    rc, _, _ = oracle.paged_attention(sc.q[0], sc.local[0], sc.staging[0], resolved, lens, sc.Hq, sc.Hkv,
                                      sc.D, sc.T, sc.sm_scale)
    assert rc == oracle.E_INVAL


def test_bf16_rounding_helper_is_nearest_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -2.5, 1.0 + 2 ** -8 + 2 ** -20, 0.0])
    ref = torch.tensor(x, dtype=torch.float64).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (oracle.to_bf16(x) == ref).all()
