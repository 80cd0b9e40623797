"""Host-side calculator for the throughput model of the paper's Sec. 3.4 (Eqs. 5-10) and for the
payload sizes of Sec. 3.3.  Closed forms only; no device work.

gamma = draft tokens per cycle, alpha = independent acceptance probability of a draft token,
t_draft / t_verify / t_rtt = time to draft gamma tokens, to verify them, and the network round
trip (serialisation included), in any one unit.
"""
from __future__ import annotations


def expected_length(alpha: float, gamma: int) -> float:
    """Eq. (5): expected tokens per cycle, (1 - alpha^gamma) / (1 - alpha); gamma at alpha = 1."""
    if not (0.0 <= alpha <= 1.0) or gamma < 1:
        raise ValueError("need 0 <= alpha <= 1 and gamma >= 1")
    if alpha == 1.0:
        return float(gamma)
    return (1.0 - alpha ** gamma) / (1.0 - alpha)


def latency_sync(t_draft: float, t_rtt: float, t_verify: float) -> float:
    """Eq. (6): one stop-and-wait cycle."""
    return t_draft + t_rtt + t_verify


def throughput_sync(alpha: float, gamma: int, t_draft: float, t_rtt: float, t_verify: float) -> float:
    """Eq. (7)."""
    return expected_length(alpha, gamma) / latency_sync(t_draft, t_rtt, t_verify)


def expected_time_async(alpha: float, gamma: int, t_draft: float, t_rtt: float, t_verify: float) -> float:
    """Eq. (9): alpha^gamma * max(t_draft, t_rtt + t_verify) + (1 - alpha^gamma) * (t_draft + t_rtt + t_verify)."""
    hit = alpha ** gamma
    return hit * max(t_draft, t_rtt + t_verify) + (1.0 - hit) * (t_draft + t_rtt + t_verify)


def throughput_async(alpha: float, gamma: int, t_draft: float, t_rtt: float, t_verify: float) -> float:
    return expected_length(alpha, gamma) / expected_time_async(alpha, gamma, t_draft, t_rtt, t_verify)


def speedup(alpha: float, gamma: int, t_draft: float, t_rtt: float, t_verify: float) -> float:
    """S = R_async / R_sync = L_sync / E[T_async] (the expected length cancels)."""
    return latency_sync(t_draft, t_rtt, t_verify) / expected_time_async(alpha, gamma, t_draft, t_rtt, t_verify)


def speedup_limit(t_draft: float, t_rtt: float, t_verify: float) -> float:
    """Eq. (10): alpha -> 1 in the compute-bound case t_draft >= t_rtt + t_verify."""
    return 1.0 + (t_rtt + t_verify) / t_draft


def downlink_bytes(k: int, fp16: bool = False, rows: int = 1) -> int:
    """Size of a wire message of `rows` full rows of k (id, prob) pairs (see picospec_wire_pack)."""
    pad4 = lambda n: (n + 3) // 4 * 4
    return 16 + pad4(2 * rows) + 4 * rows * k + pad4((2 if fp16 else 4) * rows * k)


def dense_row_bytes(vocab: int, bytes_per_prob: int = 4) -> int:
    """One full probability row, the payload the sparse message replaces."""
    return vocab * bytes_per_prob
