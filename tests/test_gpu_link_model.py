"""The paper's transparency condition with a real link (Section 2.3 / 4: a transfer of m bytes over
a link of bandwidth B is hidden while it fits in the latency window, B * L >= m), measured: the lent
arena lives in pinned host memory, so the prefetch crosses PCIe. The time per layer of the
one-launch pass must follow max(T0, m / B) within 20 % on both sides of the knee m* = B * T0, with
B and T0 measured in the same test and the knee placed by the sizing helper."""
import pytest

from paper_2609_27040_b200 import build as build_mod
from paper_2609_27040_b200 import capacity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()


def test_layer_time_follows_the_transparency_model_on_both_sides_of_the_knee():
    from paper_2609_27040_b200.microbench import link_point
    base = link_point(0.0)                         # nothing lent: T0
    far = link_point(0.05)                         # far beyond the knee: gives the link rate B
    assert base["device_status"] == 0 and far["device_status"] == 0
    t0 = base["us_per_layer"] * 1e-6
    link = far["link_gbs"] * 1e9
    size = capacity.size_from_measurement(link, t0, base["kv_bytes_per_layer"], num_groups=8)
    f_knee = size["knee_fraction_of_kv"]
    assert 0.001 < f_knee < 0.05, f_knee           # a PCIe link hides about 1 % of the KV per layer
    checked = []
    for f in (f_knee / 4, f_knee / 2, 3 * f_knee, 0.05):
        row = far if f == 0.05 else link_point(f)
        assert row["device_status"] == 0
        model = capacity.layer_time(t0, row["lent_bytes_per_layer"], link) * 1e6
        ratio = row["us_per_layer"] / model
        checked.append((round(f, 5), row["lent_bytes_per_layer"], round(row["us_per_layer"], 1), round(model, 1), round(ratio, 3)))
        assert 0.8 <= ratio <= 1.2, checked
        hidden = capacity.transfer_hidden(row["lent_bytes_per_layer"], link, t0)
        assert hidden == (row["lent_bytes_per_layer"] <= size["knee_bytes_per_layer"])
    # beyond the knee the link is the bound: the stall is what the model says, to a few per cent
    assert abs(checked[-1][4] - 1.0) < 0.1, checked
