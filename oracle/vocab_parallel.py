"""CPU statement of vocabulary-parallel verification.  TEST INFRASTRUCTURE ONLY.

The paper's verifier model runs on two to four GPUs (Sec. 4.1), so its output layer leaves the
target logits sharded along the vocabulary: rank r holds columns [v0_r, v0_r + Vs_r) of every row.
Verification (Sec. 3.3 accept test, Sec. 2.1 rule, residual resampling) then needs one exchange:

  per rank, from its slice alone
    records   per (row, 1024-entry chunk): the chunk's largest logit m_c and
              s_c = sum over the chunk of exp((l - m_c) / T)
    entries   the logits at the stored indices of the sparse draft rows and at the drafted token that
              fall into the slice (-inf for the others)
  exchange    all-gather of the records (chunks never straddle ranks: every v0_r is a multiple of
              1024), element-wise maximum of the entries (every index has one owner)
  every rank  row normaliser Z = sum_c s_c exp((m_c - m) / T), p at every gathered entry, accept
              test, residual mass R = 1 - sum_S min(p, q~), first-rejection scan, and the level-1
              pick of a chunk from the chunk masses  P_c - sum_{S in c} min(p, q~)
  the owner   of the picked chunk draws the token inside it (level 2) from its slice; element-wise
              maximum of the tokens (-1 from the other ranks)

Everything is double precision and written from the definitions; the only identity used is
sum_v max(0, p_v - q~_v) = sum_v p_v - sum_S min(p_v, q~_v), chunk by chunk.  The pin
(tests/test_oracle_pins.py) is that this reproduces the plain oracle on the concatenated vocabulary.
"""
from __future__ import annotations

import numpy as np

CHUNK = 1024
RESID_ZERO = 1e-12        # the vanished-residual reading of the plain oracle


def slice_records(slice_logits: np.ndarray, temperature: np.ndarray, chunk: int = CHUNK):
    """[B, R, Vs] fp32 slice -> (m [B,R,nc] f64, s [B,R,nc] f64): chunk maximum and
    sum exp((l - m_c)/T); an all -inf chunk has m = -inf, s = 0."""
    B, R, Vs = slice_logits.shape
    nc = (Vs + chunk - 1) // chunk
    m = np.full((B, R, nc), -np.inf)
    s = np.zeros((B, R, nc))
    for b in range(B):
        T = np.float64(temperature[b])
        for c in range(nc):
            blk = slice_logits[b, :, c * chunk:(c + 1) * chunk].astype(np.float64)
            mc = blk.max(axis=-1)
            m[b, :, c] = mc
            ok = np.isfinite(mc)
            with np.errstate(invalid="ignore"):
                e = np.exp((blk - mc[:, None]) / T)
            s[b, :, c] = np.where(ok, np.where(np.isnan(e), 0.0, e).sum(axis=-1), 0.0)
    return m, s


def slice_entries(slice_logits: np.ndarray, v0: int, draft_tok, q_idx, q_count):
    """Logits of the stored entries (slots 0..K-1) and of the drafted token (slot K) of every draft
    position that this slice holds; -inf elsewhere.  -> [B, G, K+1] f64"""
    B, R, Vs = slice_logits.shape
    G = R - 1
    K = q_idx.shape[-1]
    out = np.full((B, G, K + 1), -np.inf)
    for b in range(B):
        for i in range(G):
            n = int(q_count[b, i])
            for k in range(max(0, min(n, K))):
                v = int(q_idx[b, i, k])
                if v0 <= v < v0 + Vs:
                    out[b, i, k] = slice_logits[b, i, v - v0]
            x = int(draft_tok[b, i])
            if v0 <= x < v0 + Vs:
                out[b, i, K] = slice_logits[b, i, x - v0]
    return out


def merge_records(parts):
    """All-gather along the chunk axis: [(m, s) per rank] -> (m, s) of the whole vocabulary."""
    return np.concatenate([p[0] for p in parts], axis=-1), np.concatenate([p[1] for p in parts], axis=-1)


def merge_entries(parts):
    """Element-wise maximum over ranks."""
    out = parts[0]
    for p in parts[1:]:
        out = np.maximum(out, p)
    return out


def decide(m, s, entries, temperature, draft_tok, q_idx, q_prob, q_count, u_accept, u_resample, chunk_owner):
    """What every rank computes after the exchange.  chunk_owner[c] = rank that holds chunk c.
    -> dict(accept_len, p_draft, resid_mass, borderline_count, row [B] sampled row, use_resid [B],
            cstar [B] picked chunk (-1: nothing to draw), owner [B], Z [B], mx [B])"""
    B, R, nc = m.shape
    G = R - 1
    K = q_idx.shape[-1]
    accept_len = np.zeros(B, np.int32)
    p_draft = np.zeros((B, G))
    resid = np.zeros((B, G))
    row = np.zeros(B, np.int32)
    use_resid = np.zeros(B, bool)
    cstar = np.full(B, -1, np.int32)
    Zs, mxs = np.zeros(B), np.zeros(B)
    nborder = 0
    for b in range(B):
        T = np.float64(temperature[b])
        mx = m[b].max(axis=-1)                                            # [R]
        Z = (s[b] * np.exp((m[b] - mx[:, None]) / T)).sum(axis=-1)         # [R]
        acc = np.ones(G, bool)
        border = np.zeros(G, bool)
        pmin = [None] * G
        for i in range(G):
            n = int(q_count[b, i])
            pk = np.exp((entries[b, i, :n] - mx[i]) / T) / Z[i]
            qk = q_prob[b, i, :n].astype(np.float64)
            pmin[i] = np.minimum(pk, qk)
            resid[b, i] = max(0.0, 1.0 - pmin[i].sum())
            x = int(draft_tok[b, i])
            px = np.exp((entries[b, i, K] - mx[i]) / T) / Z[i]
            p_draft[b, i] = px
            hit = np.nonzero(q_idx[b, i, :n] == x)[0]
            if len(hit):
                qx = np.float64(q_prob[b, i, hit[0]])
                if qx > 0:
                    ratio = px / qx
                    u = np.float64(u_accept[b, i])
                    acc[i] = u < min(1.0, ratio)
                    border[i] = abs(ratio - u) <= 1e-6 * u
        a = 0
        while a < G and acc[a]:
            a += 1
        accept_len[b] = a
        nborder += int(border[:min(a, G - 1) + 1].sum()) if G > 0 else 0
        # chunk masses of the sampled row
        j = a
        row[b] = j
        P = s[b, j] * np.exp((m[b, j] - mx[j]) / T) / Z[j]                # mass of p in every chunk
        M = P.copy()
        resid_row = j < G and int(q_count[b, j]) > 0
        if resid_row:
            n = int(q_count[b, j])
            Mr = P.copy()
            np.subtract.at(Mr, q_idx[b, j, :n] // CHUNK, pmin[j])
            Mr = np.maximum(Mr, 0.0)
            if Mr.sum() > RESID_ZERO:
                M = Mr
            else:
                resid_row = False
        use_resid[b] = resid_row
        tot = M.sum()
        thr = np.float64(u_resample[b, 0]) * tot
        cum = np.cumsum(M)
        first = np.nonzero(cum > thr)[0]
        cstar[b] = first[0] if len(first) else np.nonzero(M > 0)[0][-1]
        Zs[b], mxs[b] = Z[j], mx[j]
    owner = np.asarray(chunk_owner)[cstar]
    return dict(accept_len=accept_len, p_draft=p_draft, resid_mass=resid, borderline_count=nborder, row=row,
                use_resid=use_resid, cstar=cstar, owner=owner, Z=Zs, mx=mxs)


def draw_in_slice(slice_logits, v0, rank, d, temperature, q_idx, q_prob, q_count, u_resample):
    """Level 2 by the owner of the picked chunk, from its slice.  -> token [B] (-1 where another
    rank owns the chunk)."""
    B = slice_logits.shape[0]
    tok = np.full(B, -1, np.int32)
    for b in range(B):
        if d["owner"][b] != rank:
            continue
        T = np.float64(temperature[b])
        j, c = int(d["row"][b]), int(d["cstar"][b])
        lo = c * CHUNK - v0
        blk = slice_logits[b, j, lo:lo + CHUNK].astype(np.float64)
        r = np.exp((blk - d["mx"][b]) / T) / d["Z"][b]
        if d["use_resid"][b]:
            n = int(q_count[b, j])
            q = np.zeros(len(blk))
            for k in range(n):
                v = int(q_idx[b, j, k])
                if c * CHUNK <= v < c * CHUNK + len(blk):
                    q[v - c * CHUNK] = q_prob[b, j, k]
            r = np.maximum(r - q, 0.0)
        thr = np.float64(u_resample[b, 1]) * r.sum()
        cum = np.cumsum(r)
        first = np.nonzero(cum > thr)[0]
        tok[b] = c * CHUNK + (first[0] if len(first) else np.nonzero(r > 0)[0][-1])
    return tok


def verify_sharded(slices, v0s, temperature, draft_tok, q_idx, q_prob, q_count, u_accept, u_resample):
    """The whole flow on a list of slices (one per rank).  -> dict like oracle.verify."""
    parts = [slice_records(sl, temperature) for sl in slices]
    ents = [slice_entries(sl, v0, draft_tok, q_idx, q_count) for sl, v0 in zip(slices, v0s)]
    m, s = merge_records(parts)
    entries = merge_entries(ents)
    chunk_owner = np.concatenate([np.full(p[0].shape[-1], r) for r, p in enumerate(parts)])
    d = decide(m, s, entries, temperature, draft_tok, q_idx, q_prob, q_count, u_accept, u_resample, chunk_owner)
    toks = [draw_in_slice(sl, v0, r, d, temperature, q_idx, q_prob, q_count, u_resample)
            for r, (sl, v0) in enumerate(zip(slices, v0s))]
    token = toks[0]
    for t in toks[1:]:
        token = np.maximum(token, t)
    return dict(accept_len=d["accept_len"], p_draft=d["p_draft"], resid_mass=d["resid_mass"],
                borderline_count=d["borderline_count"], token=token)
