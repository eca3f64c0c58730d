"""Pins of the capacity model against what the paper states (Section 4): Eq. 1 holds with equality
when the borrowed amounts fill the link, the slice-size formula is the largest size for which every
split of the shares stays feasible, and the layer-time model has its knee at m = B * L."""
import numpy as np

from paper_2609_27040_b200 import capacity as C


def test_eq1_equality_and_slice_capacity_is_the_largest_freely_splittable_size():
    rng = np.random.default_rng(0)
    for _ in range(200):
        B = float(rng.uniform(10, 900))            # GB/s
        Li, Lj = (float(x) for x in rng.uniform(1e-3, 5e-2, size=2))
        L = min(Li, Lj)
        total = B * L                              # m_ji + m_ij at capacity
        assert np.isclose(C.slice_capacity(B, Li, Lj), 2 * total)
        for frac in (0.0, 0.3, 0.5, 1.0):
            m_ji, m_ij = frac * total, (1 - frac) * total
            # every shift of the shares stays within the link ...
            for v in np.linspace(0, min(m_ji, m_ij), 5):       # shares stay non-negative
                assert C.shares_feasible(m_ji, m_ij, float(v), Li, Lj, B)
            # ... and with equal windows the demand is exactly the link (Eq. 1)
            assert np.isclose(C.bandwidth_demand(m_ji, L, m_ij, L), B)
        # 5 % more than the capacity: the share that sits on the shorter window breaks the bound
        big = 1.05 * total
        m_short = (big, 0.0) if Li <= Lj else (0.0, big)
        assert not C.shares_feasible(m_short[0], m_short[1], 0.0, Li, Lj, B)


def test_layer_time_knee_and_transparency():
    B, L = 51.2e9, 94.1e-6                          # the measured PCIe link and layer time of the 8B shapes
    knee = B * L
    assert abs(knee - 4.82e6) < 0.01e6
    for m in (0.0, 0.5 * knee, knee):
        assert C.transfer_hidden(m, B, L) and C.layer_time(L, m, B) == L
    for m in (1.01 * knee, 2 * knee, 25 * knee):
        assert not C.transfer_hidden(m, B, L)
        assert np.isclose(C.layer_time(L, m, B), m / B)
    # the paper's own scale: 300 GB/s links and windows of tens of milliseconds give slices of GBs
    assert np.isclose(C.slice_capacity(300e9, 20e-3, 35e-3), 12e9)


def test_appendix_a_shares_exist_exactly_below_the_link_rate():
    """Brute force over the shares alpha and beta against the closed form of Appendix A."""
    rng = np.random.default_rng(1)
    grid = np.linspace(0.0, 1.0, 401)[1:-1]
    hits = [0, 0]
    for _ in range(300):
        Li, Lj = (float(x) for x in rng.uniform(1.0, 5.0, size=2))
        Bji, Bij = (float(x) for x in rng.uniform(5.0, 10.0, size=2))
        m_ji, m_ij = (float(x) for x in rng.uniform(0.5, 25.0, size=2))
        a_ok = ((grid * Bji * Li > m_ji) & ((1 - grid) * Bji * Lj > m_ij)).any()      # (1) and (4)
        b_ok = (((1 - grid) * Bij * Li > m_ji) & (grid * Bij * Lj > m_ij)).any()      # (3) and (2)
        demand = C.bandwidth_demand(m_ji, Li, m_ij, Lj)
        if abs(demand - min(Bji, Bij)) / min(Bji, Bij) < 0.02:
            continue                                     # too close to the boundary for a grid of shares
        want = C.split_exists(m_ji, m_ij, Li, Lj, Bji, Bij)
        assert bool(a_ok and b_ok) == want
        hits[int(want)] += 1
    assert min(hits) > 30


def test_reclaim_release_rule_and_window_fraction():
    assert C.release_on_reclaim(8.0) == (4.0, 4.0)          # r = 2: k/2 on each side
    remote, local = C.release_on_reclaim(9.0, 3.0)
    assert np.isclose(remote + local, 9.0) and np.isclose(local, 2 * remote)   # (r - 1) * k of local data goes with k remote
    assert C.window_fraction(32) == 31 / 32 and C.window_fraction(8) == 7 / 8 and C.window_fraction(8) < C.window_fraction(32)
    s = C.size_from_measurement(51.2e9, 94.1e-6, 614.3e6, num_groups=32)
    assert abs(s["knee_fraction_of_kv"] - 0.00784) < 1e-4
    assert np.isclose(s["window_seconds"], 31 * 94.1e-6) and np.isclose(s["slice_bytes"], 2 * 51.2e9 * 31 * 94.1e-6)
