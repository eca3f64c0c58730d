"""The layer-dependent form of the one-launch pass (slice_step_begin): the queries of layer l+1 are
released to the running kernel only after the output of layer l is complete, as in a decoder, where
they are computed from it. Here they ARE that output (copied, negated, or aliased in memory), so a
layer that started before its queries had arrived, or queries released before the output they come
from was complete, would attend to the wrong rows and disagree with the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_27040_b200 import binding as B
from paper_2609_27040_b200 import build as build_mod
from paper_2609_27040_b200 import synth
from tests.helpers import Scenario, attention_close

pytestmark = pytest.mark.gpu

ATOL = RTOL = 1e-2


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _feed(s, L, caller, make_q=None):
    """The caller's side of a pass: release q[0]; then for every layer wait for its output, derive the
    next layer's queries from it on the caller's stream and release them."""
    assert s.slice_step_submit_q(0, caller) == B.OK
    for l in range(L - 1):
        assert s.slice_step_wait_out(l, caller) == B.OK
        if make_q is not None:
            with torch.cuda.stream(caller):
                make_q(l)
        assert s.slice_step_submit_q(l + 1, caller) == B.OK
    assert s.slice_step_wait_out(L - 1, caller) == B.OK


def test_all_queries_released_at_once_and_every_output_announced():
    """The simplest use: every layer's queries exist beforehand and are released right after the pass
    has begun; the caller's stream then waits for the announcement of every layer's output, last
    layer first (all of them are set by the time the launch has ended)."""
    from tests.gpu_helpers import GpuScenario
    wl = synth.Workload("dep0", 4, 16, 4, 5, 60, 900, 0.4)
    sc = Scenario(wl, 5)
    g = GpuScenario(sc, decode_ctas=10)
    seqs = np.asarray(sc.seq_ids, np.int32)
    caller = torch.cuda.Stream()
    q = g.q.view(torch.bfloat16)
    out = torch.zeros_like(q)
    assert g.s.slice_step_begin(seqs, q, sc.Hq, float(sc.sm_scale), out, True, g.main) == B.OK
    for layer in range(sc.L):
        assert g.s.slice_step_submit_q(layer, caller) == B.OK
    for layer in reversed(range(sc.L)):
        assert g.s.slice_step_wait_out(layer, caller) == B.OK
    caller.synchronize()                                        # returns only when every output was announced
    assert g.s.slice_stats()["device_status"] == 0
    torch.cuda.synchronize()
    g.device_ok()
    for layer in range(sc.L):
        rc, resolved, k = sc.orc.gather(layer, sc.seq_ids, sc.lent, sc.staging)
        _, ref, _ = oracle.paged_attention(sc.q[layer], sc.local[layer], sc.staging[layer % wl.ring_slots], resolved,
                                           sc.lengths(), sc.Hq, sc.Hkv, sc.D, sc.T, sc.sm_scale)
        assert attention_close(out[layer].double().cpu().numpy(), ref, ATOL, RTOL)[0], layer


@pytest.mark.parametrize("static", [0, 1])
def test_queries_released_layer_by_layer_small(static):
    from tests.gpu_helpers import GpuScenario
    wl = synth.Workload("dep", 6, 32, 8, 7, 100, 1200, 0.4)
    sc = Scenario(wl, 13)
    g = GpuScenario(sc, decode_ctas=12, static_split=static)
    seqs = np.asarray(sc.seq_ids, np.int32)
    caller = torch.cuda.Stream()
    for rep in range(2):
        q = g.q.view(torch.bfloat16).clone()
        q[1:] = 0                                               # later layers' queries do not exist yet
        out = torch.zeros_like(q)
        torch.cuda.synchronize()
        assert g.s.slice_step_begin(seqs, q, sc.Hq, float(sc.sm_scale), out, True, g.main) == B.OK
        rc, q_ready, out_ready, epoch = g.s.slice_step_flags()
        assert rc == B.OK and q_ready and out_ready and epoch == rep + 1
        _feed(g.s, sc.L, caller, lambda l: q[l + 1].copy_(out[l]))
        torch.cuda.synchronize()
        g.device_ok()
        for layer in range(sc.L):
            if layer:
                assert torch.equal(q[layer], out[layer - 1])
            rc, resolved, k = sc.orc.gather(layer, sc.seq_ids, sc.lent, sc.staging)
            _, ref, _ = oracle.paged_attention(_bits(q[layer]), sc.local[layer], sc.staging[layer % wl.ring_slots], resolved,
                                               sc.lengths(), sc.Hq, sc.Hkv, sc.D, sc.T, sc.sm_scale)
            ok, max_abs, _ = attention_close(out[layer].double().cpu().numpy(), ref, ATOL, RTOL)
            assert ok, (rep, layer, max_abs)
    # a free-running pass afterwards is not disturbed by the flags the dependent passes left
    g.out.zero_()
    assert g.s.slice_decode_step(seqs, g.q, sc.Hq, float(sc.sm_scale), g.out, False, True, g.main, g.side) == B.OK
    torch.cuda.synchronize()
    g.device_ok()
    got = g.out.view(torch.bfloat16).double().cpu().numpy()
    for layer in range(sc.L):
        rc, resolved, k = sc.orc.gather(layer, sc.seq_ids, sc.lent, sc.staging)
        _, ref, _ = oracle.paged_attention(sc.q[layer], sc.local[layer], sc.staging[layer % wl.ring_slots], resolved,
                                           sc.lengths(), sc.Hq, sc.Hkv, sc.D, sc.T, sc.sm_scale)
        assert attention_close(got[layer], ref, ATOL, RTOL)[0]


@pytest.mark.parametrize("ctas,how", [(0, "alias"), (140, "kernel"), (147, "relay")])
def test_queries_released_layer_by_layer_full_batch(ctas, how):
    """The benchmark's batch on 6 layers. 'alias': one CTA per SM (no room for any other kernel), the
    next layer's queries are the previous layer's output in place (q = X[l], out = X[l+1]), so the
    caller only waits and releases. 'kernel': 140 CTAs, the caller's own kernel (an elementwise
    negation, launched once beforehand so that its code is loaded) computes the next queries on the
    SMs left free while the pass runs. 'relay': 147 CTAs and the library's one-thread relay kernel on
    the SM left free, which hands every layer's output over as the next layer's queries (aliased as
    in 'alias') through the device words themselves instead of stream-ordered operations."""
    from tests.test_gpu_full_batch import FullBatch
    L = 6
    fb = FullBatch("llama3_8b_decode", L, decode_ctas=ctas)
    wl = fb.wl
    caller = torch.cuda.Stream()
    if how in ("alias", "relay"):
        X = torch.zeros((L + 1,) + tuple(fb.q.shape[1:]), device="cuda", dtype=torch.bfloat16)
        X[0].copy_(fb.q[0])
        q, out, make_q = X[:L], X[1:], None
    else:
        q = fb.q.clone()
        q[1:] = 0
        out = torch.zeros_like(q)
        make_q = lambda l: torch.neg(out[l], out=q[l + 1])
        make_q(0)                     # first launch: loads the kernel's code, which cannot finish beside a running pass
        q[1] = 0
    torch.cuda.synchronize()
    for rep in range(2):
        assert fb.s.slice_step_begin(fb.seqs, q, wl.num_q_heads, fb.scale, out, True, fb.main) == B.OK
        if how == "relay":
            assert fb.s.slice_step_relay(caller) == B.OK
        else:
            _feed(fb.s, L, caller, make_q)
        torch.cuda.synchronize()
        st = fb.s.slice_stats()
        assert st["device_status"] == 0 and st["last_cuda_error"] == 0
    resolved, k = fb.check_tables()
    for layer in range(L):
        if layer and how == "kernel":
            assert torch.equal(q[layer], -out[layer - 1])
        fb.check_attention_in_full(layer, resolved, k, q_layer=q[layer], out_layer=out[layer])
    fb.s.close()
