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
