"""The paper's capacity model for a memory slice (Section 4, Eq. 1 and the slice-size formula):
closed forms only, used by the link microbenchmark to place the knee and by tests as pins. Units are
free as long as they agree (bytes, bytes per second, seconds)."""
from __future__ import annotations


def transfer_hidden(m: float, bandwidth: float, window: float) -> bool:
    """A transfer of m over a link of the given bandwidth is transparent when it completes inside
    the latency window between two uses of the data: bandwidth * window >= m (Section 4)."""
    return bandwidth * window >= m


def layer_time(t0: float, m: float, bandwidth: float) -> float:
    """Time per layer when m bytes must cross the link for every layer that takes t0 to compute:
    the transfer is hidden until it no longer fits, then it is the bound."""
    return max(t0, m / bandwidth)


def bandwidth_demand(m_ji: float, window_i: float, m_ij: float, window_j: float) -> float:
    """Left-hand side of Eq. 1: link bandwidth needed so that GPU i cycles through the m_ji it
    borrowed within its window and GPU j through its m_ij within its own."""
    return m_ji / window_i + m_ij / window_j


def shares_feasible(m_ji: float, m_ij: float, m_v: float, window_i: float, window_j: float, bandwidth: float) -> bool:
    """The generalisation of Eq. 1 to shares that move by m_v in either direction
    (0 <= m_v <= m_ji + m_ij): both shifted demands must stay within the link."""
    return (bandwidth_demand(m_ji - m_v, window_i, m_ij + m_v, window_j) <= bandwidth * (1 + 1e-12) and
            bandwidth_demand(m_ji + m_v, window_i, m_ij - m_v, window_j) <= bandwidth * (1 + 1e-12))


def slice_capacity(bandwidth: float, window_i: float, window_j: float) -> float:
    """Largest slice whose shares can move freely: 2 * B * min(L_i, L_j) (expansion ratio 2: both GPUs
    contribute as much as the pair borrows)."""
    return 2.0 * bandwidth * min(window_i, window_j)


def split_exists(m_ji: float, m_ij: float, window_i: float, window_j: float, b_ji: float, b_ij: float) -> bool:
    """Appendix A: each direction of the link is divided between the two GPUs (shares alpha and
    1 - alpha of the j->i direction, beta and 1 - beta of i->j), and each GPU must be able to bring
    in and send out what it borrowed within its own window (inequalities (1)-(4), strict). Shares
    that satisfy all four exist exactly when m_ji / L_i + m_ij / L_j is below both directions'
    bandwidth."""
    return bandwidth_demand(m_ji, window_i, m_ij, window_j) < min(b_ji, b_ij)


def release_on_reclaim(k: float, expansion_ratio: float = 2.0):
    """Section 4.1: when the lender takes k back from the borrower's remote data, the
    (r - 1) * k of local data of the same requests (their other layers) is useless and goes too.
    With the expansion ratio fixed at 2 both amounts are equal, and a reclaim of k in total frees
    k / 2 on each side. Returns (remote released, local released) for a reclaim of k in total."""
    remote = k / expansion_ratio
    return remote, (expansion_ratio - 1.0) * remote


def window_fraction(num_groups: int) -> float:
    """Section 4.2.2: the effective latency window is proportional to (k - 1) / k for k units in the
    cycle (layers, or layer groups once layers are grouped), so fewer, larger groups shrink it."""
    return (num_groups - 1) / num_groups


def size_from_measurement(link_bytes_per_s: float, layer_seconds: float, kv_bytes_per_layer: float,
                          num_groups: int = 0) -> dict:
    """Sizing from measured figures: a link rate B, the time T0 one layer (or layer group) takes to
    compute with nothing lent, and the KV bytes a layer reads. The latency window of a layer's data
    is the rest of the cycle, (k - 1) / k of the pass for k units; per unit of the cycle the link
    can hide B * T0 bytes (the knee of layer_time). Returns the knee in bytes per layer and as a
    fraction of the layer's KV, and the slice size 2 * B * L of Section 4.1 for the pass as window."""
    knee = link_bytes_per_s * layer_seconds
    out = {"knee_bytes_per_layer": knee, "knee_fraction_of_kv": knee / kv_bytes_per_layer}
    if num_groups:
        window = window_fraction(num_groups) * num_groups * layer_seconds
        out["window_seconds"] = window
        out["slice_bytes"] = slice_capacity(link_bytes_per_s, window, window)
    return out
