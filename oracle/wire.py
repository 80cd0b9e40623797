"""CPU oracle for the wire format of sparse rows (Sec. 3.3: the verifier sends "(id, prob)" pairs,
under 100 bytes for K = 10, laid out so that the receiver can view the arrays in place) and for
the throughput model of Sec. 3.4 (Eqs. 5-10).

TEST INFRASTRUCTURE ONLY, like the rest of this package.  Plain numpy / Python, written from the
definitions: the message layout below and the sums and case analysis of Sec. 3.4 as printed (the
closed forms are what the product's calculator uses; here the sums are taken term by term).

Message layout (little endian):
    0   u32  magic 0x31505350 ("PSP1")
    4   u32  R, the number of rows
    8   u16  K, the capacity of a dense row
    10  u16  probability type: 0 = fp32, 1 = fp16 (round to nearest even)
    12  u32  N = sum over rows of max(count, 0)
    16  i16  count[R]   (-1 = invalid row), zero-padded to a multiple of 4 bytes
    ..  i32  id[N]      rows in order, entries in stored order
    ..  prob[N]         fp32 or fp16; the message is zero-padded to a multiple of 4 bytes
"""
from __future__ import annotations

import numpy as np

MAGIC = 0x31505350
F32, F16 = 0, 1


def _pad4(n: int) -> int:
    return (n + 3) // 4 * 4


def wire_size(rows: int, entries: int, prob_type: int) -> int:
    return 16 + _pad4(2 * rows) + 4 * entries + _pad4((4 if prob_type == F32 else 2) * entries)


def pack(q_idx, q_prob, q_count, prob_type: int = F32) -> np.ndarray:
    q_idx = np.asarray(q_idx, np.int32)
    q_prob = np.asarray(q_prob, np.float32)
    q_count = np.asarray(q_count, np.int32).reshape(-1)
    K = q_idx.shape[-1]
    q_idx = q_idx.reshape(-1, K)
    q_prob = q_prob.reshape(-1, K)
    R = q_idx.shape[0]
    q_count = np.where((q_count > K) | (q_count < -1), -1, q_count).astype(np.int32)   # bad count: the row travels as invalid
    ids, probs = [], []
    for r in range(R):
        n = max(int(q_count[r]), 0)
        ids.append(q_idx[r, :n])
        probs.append(q_prob[r, :n])
    ids = np.concatenate(ids) if ids else np.zeros(0, np.int32)
    probs = np.concatenate(probs) if probs else np.zeros(0, np.float32)
    N = ids.size
    out = np.zeros(wire_size(R, N, prob_type), np.uint8)
    out[0:4] = np.array([MAGIC], "<u4").view(np.uint8)
    out[4:8] = np.array([R], "<u4").view(np.uint8)
    out[8:10] = np.array([K], "<u2").view(np.uint8)
    out[10:12] = np.array([prob_type], "<u2").view(np.uint8)
    out[12:16] = np.array([N], "<u4").view(np.uint8)
    o = 16
    out[o:o + 2 * R] = q_count.astype("<i2").view(np.uint8)
    o += _pad4(2 * R)
    out[o:o + 4 * N] = ids.astype("<i4").view(np.uint8)
    o += 4 * N
    if prob_type == F32:
        out[o:o + 4 * N] = probs.astype("<f4").view(np.uint8)
    else:
        out[o:o + 2 * N] = probs.astype("<f2").view(np.uint8)
    return out


def unpack(buf: np.ndarray, rows: int, K: int):
    """Dense (q_idx [R,K] i32 padded with -1, q_prob [R,K] f32 padded with 0, q_count [R] i32).
    A message that does not match (rows, K) or is malformed gives all rows invalid (-1, 0, -1)."""
    buf = np.asarray(buf, np.uint8)
    bad = (np.full((rows, K), -1, np.int32), np.zeros((rows, K), np.float32), np.full((rows,), -1, np.int32))
    if buf.size < 16:
        return bad
    magic, R = (int(x) for x in buf[0:8].view("<u4"))
    Kh, ptype = (int(x) for x in buf[8:12].view("<u2"))
    N = int(buf[12:16].view("<u4")[0])
    if magic != MAGIC or R != rows or Kh != K or ptype not in (F32, F16) or buf.size < wire_size(R, N, ptype):
        return bad
    o = 16
    counts = buf[o:o + 2 * R].view("<i2").astype(np.int32)
    if np.any(counts > K) or np.any(counts < -1) or int(np.maximum(counts, 0).sum()) != N:
        return bad
    o += _pad4(2 * R)
    ids = buf[o:o + 4 * N].view("<i4")
    o += 4 * N
    probs = buf[o:o + 4 * N].view("<f4") if ptype == F32 else buf[o:o + 2 * N].view("<f2").astype(np.float32)
    q_idx, q_prob, q_count = bad[0].copy(), bad[1].copy(), counts.copy()
    p = 0
    for r in range(R):
        n = max(int(counts[r]), 0)
        q_idx[r, :n] = ids[p:p + n]
        q_prob[r, :n] = probs[p:p + n]
        p += n
    return q_idx, q_prob, q_count


# ---- Sec. 3.4: the throughput model, term by term ------------------------------------------------

def expected_length(alpha: float, gamma: int) -> float:
    """Eq. (5): L = number of tokens a cycle yields, 1 <= L <= gamma; L = k < gamma when the first
    k - 1 ... are accepted; written as the expectation of the truncated geometric variable."""
    # P(L >= k) = alpha^(k-1) for k = 1 .. gamma, and E[L] = sum_k P(L >= k)
    return float(sum(alpha ** (k - 1) for k in range(1, gamma + 1)))


def latency_sync(t_draft: float, t_rtt: float, t_verify: float) -> float:
    """Eq. (6)."""
    return t_draft + t_rtt + t_verify


def throughput_sync(alpha, gamma, t_draft, t_rtt, t_verify) -> float:
    """Eq. (7)."""
    return expected_length(alpha, gamma) / latency_sync(t_draft, t_rtt, t_verify)


def expected_time_async(alpha, gamma, t_draft, t_rtt, t_verify) -> float:
    """Eqs. (8)-(9): full hit with probability alpha^gamma costs max(T_draft, T_RTT + T_verify);
    a miss costs the synchronous latency."""
    p_hit = alpha ** gamma
    t_hit = max(t_draft, t_rtt + t_verify)
    t_miss = latency_sync(t_draft, t_rtt, t_verify)
    return p_hit * t_hit + (1.0 - p_hit) * t_miss


def throughput_async(alpha, gamma, t_draft, t_rtt, t_verify) -> float:
    return expected_length(alpha, gamma) / expected_time_async(alpha, gamma, t_draft, t_rtt, t_verify)


def speedup(alpha, gamma, t_draft, t_rtt, t_verify) -> float:
    """S = R_async / R_sync."""
    return throughput_async(alpha, gamma, t_draft, t_rtt, t_verify) / throughput_sync(alpha, gamma, t_draft, t_rtt, t_verify)
