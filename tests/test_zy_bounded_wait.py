"""The failure path of the bounded device-side waits, exercised without any fault: a wait is made to run
out (nothing ever sets the flag it polls), the kernel gives up in bounded time and reports it, and
the context stays usable."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_27040_b200 import binding as B
from paper_2609_27040_b200 import synth
from tests.gpu_helpers import GpuScenario
from tests.helpers import Scenario, attention_close

pytestmark = pytest.mark.gpu


def test_bounded_wait_expires_and_is_reported():
    """Failure path without a fault: the arrival flags of the streamed queries are withheld (test
    hook), so the kernel's wait for them runs out after about two seconds; every role gives up in
    bounded time, the launch ends, slice_stats reports SLICE_ETIMEOUT, and the context stays usable:
    a fresh slice on the same arenas decodes correctly afterwards."""
    import time
    wl = synth.Workload("timeout", 2, 8, 4, 3, 40, 200, 0.4)
    sc = Scenario(wl, 41)
    g = GpuScenario(sc, decode_ctas=4, flags=B.FLAG_TEST_WITHHOLD_Q)
    seqs = np.array(sc.seq_ids, np.int32)
    qh = g.q.cpu().pin_memory()
    oh = torch.zeros_like(qh).pin_memory()
    t0 = time.perf_counter()
    assert g.s.slice_decode_step(seqs, qh, sc.Hq, float(sc.sm_scale), oh, True, True, g.main, g.side) == B.OK
    torch.cuda.synchronize()
    elapsed = time.perf_counter() - t0
    st = g.s.slice_stats()
    assert st["device_status"] == B.ETIMEOUT and st["last_cuda_error"] == 0
    assert 1.0 < elapsed < 30.0
    g.s.slice_destroy()
    g2 = GpuScenario(sc, decode_ctas=4)
    assert g2.s.slice_decode_step(seqs, qh, sc.Hq, float(sc.sm_scale), oh, True, True, g2.main, g2.side) == B.OK
    torch.cuda.synchronize()
    g2.device_ok()
    got = oh.view(torch.bfloat16).double().numpy()
    for layer in range(sc.L):
        rc, resolved, k = sc.orc.gather(layer, sc.seq_ids, sc.lent, sc.staging)
        _, ref, _ = oracle.paged_attention(sc.q[layer], sc.local[layer], sc.staging[layer % wl.ring_slots], resolved,
                                           sc.lengths(), sc.Hq, sc.Hkv, sc.D, sc.T, sc.sm_scale)
        assert attention_close(got[layer], ref, 1e-2, 1e-2)[0]
