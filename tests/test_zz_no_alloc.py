"""paged_decode_noalloc: the attention entry point for callers that must not allocate device memory
(a server whose KV-cache pool already owns the whole GPU, a decode loop that cannot take the
device-wide synchronisation of an allocation, code barred from allocator calls after start-up).

Its output is checked against the CPU oracle and against the allocating entry point, on calls in a
row that share the static scratch array, and the GPU's free memory is checked to be the same before
and after the first call that follows slice_create.

The file is named so that pytest collects it last: a run that stops at the first failure has then
already run every other test. It passes alone in a fresh process (slice_create does the one-time
set-up of the static array on the device) and after the other tests.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_27040_b200 import binding as B
from paper_2609_27040_b200 import build as build_mod
from paper_2609_27040_b200 import synth
from tests.helpers import Scenario, attention_close

pytestmark = pytest.mark.gpu

ATOL = RTOL = 1e-2   # the attention tolerance used by the parity tests


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()


def _f64(t):
    return t.view(torch.bfloat16).double().cpu().numpy()


def _oracle_layer(sc, layer, seqs, q_bits):
    """fp64 attention of `seqs` (a sub-batch, in this order) for `layer`, from the oracle's own gather."""
    rc, resolved, k = sc.orc.gather(layer, seqs, sc.lent, sc.staging)
    assert rc == oracle.OK
    lens = np.asarray([int(sc.pl.lengths[i]) for i in seqs], np.uint32)
    rc, ref, ref_lse = oracle.paged_attention(q_bits, sc.local[layer], sc.staging[layer % sc.wl.ring_slots], resolved, lens,
                                              sc.Hq, sc.Hkv, sc.D, sc.T, sc.sm_scale)
    assert rc == oracle.OK
    return ref, ref_lse


@pytest.mark.parametrize("wl", [synth.Workload("na4", 2, 32, 8, 6, 30, 700, 0.4),
                                synth.Workload("na1", 1, 8, 8, 4, 100, 500, 0.25)])
def test_noalloc_matches_oracle_and_paged_decode_twice_in_a_row(wl):
    """Two consecutive calls through the C ABI share the static scratch; each must reproduce the
    oracle's result, and that of the allocating entry point, on the same inputs. The first call
    after slice_create must leave the GPU's free memory as it found it."""
    from tests.gpu_helpers import GpuScenario
    sc = Scenario(wl, 21)
    g = GpuScenario(sc)
    first = True
    for layer in range(sc.L):
        assert g.s.prefetch_layer(layer, sc.seq_ids, g.side) == B.OK
        q2 = g.q[layer].flip(0).contiguous()          # the second call attends to a different query
        ref = torch.zeros_like(g.q[layer])
        ref_lse = torch.zeros((sc.nseq, sc.Hq), dtype=torch.float32, device="cuda")
        ref2, ref2_lse = torch.zeros_like(ref), torch.zeros_like(ref_lse)
        outs = [torch.zeros_like(ref), torch.zeros_like(ref)]
        lses = [torch.zeros_like(ref_lse), torch.zeros_like(ref_lse)]
        torch.cuda.synchronize()
        for call, q in enumerate((g.q[layer], q2)):
            free_before = torch.cuda.mem_get_info()[0]
            assert g.s.paged_decode_noalloc(layer, sc.seq_ids, q, sc.Hq, float(sc.sm_scale), outs[call], lses[call],
                                            g.main) == B.OK
            if first:                                  # nothing was allocated, by the call or by the driver under it
                torch.cuda.synchronize()
                assert torch.cuda.mem_get_info()[0] == free_before
                first = False
        assert g.s.paged_decode(layer, sc.seq_ids, g.q[layer], sc.Hq, float(sc.sm_scale), ref, ref_lse, g.main) == B.OK
        assert g.s.paged_decode(layer, sc.seq_ids, q2, sc.Hq, float(sc.sm_scale), ref2, ref2_lse, g.main) == B.OK
        torch.cuda.synchronize()
        g.device_ok()
        q_bits = (sc.q[layer], np.ascontiguousarray(sc.q[layer][::-1]))
        for call in range(2):
            want, want_lse = _oracle_layer(sc, layer, sc.seq_ids, q_bits[call])
            ok, max_abs, _ = attention_close(_f64(outs[call]), want, ATOL, RTOL)
            assert ok, max_abs
            assert np.abs(lses[call].double().cpu().numpy() - want_lse).max() <= 1e-3
            other, other_lse = (ref, ref_lse) if call == 0 else (ref2, ref2_lse)
            ok, max_abs, _ = attention_close(_f64(outs[call]), _f64(other), ATOL, RTOL)
            assert ok, max_abs
            assert np.abs(lses[call].cpu().numpy() - other_lse.cpu().numpy()).max() <= 1e-3


def test_noalloc_small_batch_after_a_large_one_reads_nothing_stale():
    """A large batch fills many partial rows and counters of the static array; the next call is a
    smaller batch of other sequences in another order, with another slot layout. Its result must be
    the oracle's: nothing the earlier call left behind may be read."""
    from tests.gpu_helpers import GpuScenario
    wl = synth.Workload("na_mix", 1, 32, 8, 12, 20, 2500, 0.4)
    sc = Scenario(wl, 27)
    g = GpuScenario(sc)
    ids = list(sc.seq_ids)
    pos = {i: n for n, i in enumerate(ids)}
    batches = [ids, [ids[7], ids[2]], ids[::-1][:5], [ids[3]], ids]
    for bt in batches:
        rows = torch.tensor([pos[i] for i in bt], device="cuda")
        q = g.q[0].index_select(0, rows).contiguous()
        out = torch.zeros_like(q)
        lse = torch.zeros((len(bt), sc.Hq), dtype=torch.float32, device="cuda")
        assert g.s.prefetch_layer(0, bt, g.side) == B.OK
        assert g.s.paged_decode_noalloc(0, bt, q, sc.Hq, float(sc.sm_scale), out, lse, g.main) == B.OK
        torch.cuda.synchronize()
        g.device_ok()
        want, want_lse = _oracle_layer(sc, 0, bt, np.ascontiguousarray(sc.q[0][[pos[i] for i in bt]]))
        ok, max_abs, _ = attention_close(_f64(out), want, ATOL, RTOL)
        assert ok, (bt, max_abs)
        assert np.abs(lse.double().cpu().numpy() - want_lse).max() <= 1e-3


def test_noalloc_rejects_batches_beyond_the_static_array():
    """260 one-block sequences x 64 query heads need 260 * 64 * 528 B > 8 MiB of partials."""
    from tests.gpu_helpers import GpuScenario
    wl = synth.Workload("na_big", 1, 64, 8, 260, 1, 16, 0.0)
    sc = Scenario(wl, 3, slack=4)
    g = GpuScenario(sc)
    out = torch.zeros_like(g.q[0])
    before = g.s.slice_stats()["kernel_launches"]
    assert g.s.paged_decode_noalloc(0, sc.seq_ids, g.q[0], sc.Hq, float(sc.sm_scale), out, None, g.main) == B.ESCRATCH
    assert g.s.slice_stats()["kernel_launches"] == before
    assert "static scratch" in B.slice_strerror(B.ESCRATCH)
    # the allocating entry point still serves the same batch
    assert g.s.paged_decode(0, sc.seq_ids, g.q[0], sc.Hq, float(sc.sm_scale), out, None, g.main) == B.OK
    torch.cuda.synchronize()
    g.device_ok()
