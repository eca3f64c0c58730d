"""paged_decode_noalloc: the attention entry point for callers that must not allocate device memory
(a server whose KV-cache pool already owns the whole GPU, a decode loop that cannot take the
device-wide synchronisation of an allocation, code barred from allocator calls after start-up).

The file is named so that pytest collects it last: a run that stops at the first failure has then
already run every other test. It passes alone in a fresh process (the first call on the device does
the one-time look-up of the static array's address) and after the other tests.
"""
import numpy as np
import pytest
import torch

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


@pytest.mark.parametrize("wl", [synth.Workload("na4", 2, 32, 8, 6, 30, 700, 0.4),
                                synth.Workload("na1", 1, 8, 8, 4, 100, 500, 0.25)])
def test_noalloc_matches_paged_decode_twice_in_a_row(wl):
    """Two consecutive calls through the C ABI share the static scratch; each must reproduce the
    result of the allocating entry point on the same inputs."""
    from tests.gpu_helpers import GpuScenario
    sc = Scenario(wl, 21)
    g = GpuScenario(sc)
    for layer in range(sc.L):
        assert g.s.prefetch_layer(layer, sc.seq_ids, g.side) == B.OK
        ref = torch.zeros_like(g.q[layer])
        ref_lse = torch.zeros((sc.nseq, sc.Hq), dtype=torch.float32, device="cuda")
        assert g.s.paged_decode(layer, sc.seq_ids, g.q[layer], sc.Hq, float(sc.sm_scale), ref, ref_lse, g.main) == B.OK
        outs, lses = [], []
        for call in range(2):
            out = torch.zeros_like(ref)
            lse = torch.zeros_like(ref_lse)
            # the second call attends to a different query, so stale scratch contents would show
            q = g.q[layer] if call == 0 else g.q[layer].flip(0).contiguous()
            assert g.s.paged_decode_noalloc(layer, sc.seq_ids, q, sc.Hq, float(sc.sm_scale), out, lse, g.main) == B.OK
            outs.append(out)
            lses.append(lse)
        ref2 = torch.zeros_like(ref)
        ref2_lse = torch.zeros_like(ref_lse)
        assert g.s.paged_decode(layer, sc.seq_ids, g.q[layer].flip(0).contiguous(), sc.Hq, float(sc.sm_scale), ref2,
                                ref2_lse, g.main) == B.OK
        torch.cuda.synchronize()
        g.device_ok()
        for got, want, got_lse, want_lse in ((outs[0], ref, lses[0], ref_lse), (outs[1], ref2, lses[1], ref2_lse)):
            ok, max_abs, _ = attention_close(_f64(got), _f64(want), ATOL, RTOL)
            assert ok, max_abs
            assert np.abs(got_lse.cpu().numpy() - want_lse.cpu().numpy()).max() <= 1e-3


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
