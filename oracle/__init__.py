"""Python face of the CPU oracle (``picospec_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's
CPU-baseline leg use this; the product package never imports it.  The wrapper
only marshals numpy arrays into the C functions; all arithmetic is in the C file.

bf16 logits are widened to fp32 by the caller (exact), the oracle widens fp32 to
double (exact), so oracle and GPU consume the same input bits.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "picospec_oracle.c")
_LIB = os.path.join(_HERE, "libpicospec_oracle.so")

CHUNK = 1024  # vocabulary entries per level-1 chunk of the two-level inverse CDF


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (IEEE semantics: no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        # a test that plants a mistake points this at its own build of a modified copy
        _lib = ctypes.CDLL(os.environ.get("PICOSPEC_ORACLE_LIB") or build())
        for name in ("pso_compress", "pso_verify", "pso_residual_sample", "pso_target_topk",
                     "pso_edge_resample", "pso_verify_range"):
            getattr(_lib, name).restype = ctypes.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _rows(logits: np.ndarray):
    assert logits.ndim == 3 and logits.dtype == np.float32 and logits.flags.c_contiguous
    return logits.shape


def cores() -> int:
    return os.cpu_count() or 1


def compress(draft_logits, temperature, top_k: int, top_p: float, k_max: int,
             u_draft=None, nthreads: int = 1):
    """draft_logits fp32 [B, G, V] -> (q_idx [B,G,k_max] i32, q_prob f32, q_count [B,G] i32,
    draft_tok [B,G] i32 or None)."""
    l = _f32(draft_logits)
    B, G, V = _rows(l)
    T = _f32(temperature)
    assert T.shape == (B,)
    q_idx = np.empty((B, G, k_max), np.int32)
    q_prob = np.empty((B, G, k_max), np.float32)
    q_count = np.empty((B, G), np.int32)
    u = tok = None
    if u_draft is not None:
        u = _f32(u_draft)
        assert u.shape == (B, G)
        tok = np.empty((B, G), np.int32)
    rc = _load().pso_compress(_p(l), ctypes.c_long(B), ctypes.c_long(G), ctypes.c_long(V),
                              ctypes.c_long(V), _p(T), ctypes.c_int(top_k),
                              ctypes.c_float(top_p), ctypes.c_int(k_max), _p(q_idx), _p(q_prob),
                              _p(q_count), _p(u), _p(tok), ctypes.c_int(nthreads))
    if rc != 0:
        raise ValueError(f"pso_compress failed: {rc}")
    return q_idx, q_prob, q_count, tok


def verify(target_logits, temperature, draft_tok, q_idx, q_prob, q_count, u_accept,
           u_resample=None, chunk: int = CHUNK, nthreads: int = 1):
    """target_logits fp32 [B, G+1, V] -> dict(accept_len [B] i32, p_draft [B,G] f64,
    resid_mass [B,G] f64, borderline_seq [B] i64, borderline_count int, token [B] i32 or None)."""
    l = _f32(target_logits)
    B, G1, V = _rows(l)
    G = G1 - 1
    T = _f32(temperature)
    tok_in = _i32(draft_tok).reshape(B, G)
    qi = _i32(q_idx)
    qp = _f32(q_prob)
    qc = _i32(q_count).reshape(B, G)
    k_max = qi.shape[-1] if qi.ndim == 3 else 1
    assert qi.shape == (B, G, k_max) and qp.shape == (B, G, k_max)
    ua = _f32(u_accept).reshape(B, G)
    accept_len = np.empty((B,), np.int32)
    p_draft = np.empty((B, G), np.float64)
    resid = np.empty((B, G), np.float64)
    border = np.zeros((B,), np.int64)
    ur = token = None
    if u_resample is not None:
        ur = _f32(u_resample)
        assert ur.shape == (B, 2)
        token = np.empty((B,), np.int32)
    rc = _load().pso_verify(_p(l), ctypes.c_long(B), ctypes.c_long(G), ctypes.c_long(V),
                            ctypes.c_long(V), _p(T), _p(tok_in), _p(qi), _p(qp), _p(qc),
                            ctypes.c_int(k_max), _p(ua), _p(accept_len), _p(p_draft), _p(resid),
                            _p(border), _p(ur), _p(token), ctypes.c_long(chunk),
                            ctypes.c_int(nthreads))
    if rc != 0:
        raise ValueError(f"pso_verify failed: {rc}")
    return {"accept_len": accept_len, "p_draft": p_draft, "resid_mass": resid,
            "borderline_seq": border, "borderline_count": int(border.sum()), "token": token}


def verify_range(target_logits, temperature, gamma, r0: int, r1: int, state_in, draft_tok, q_idx, q_prob,
                 q_count, u_accept, u_resample, out=None, chunk: int = CHUNK, nthreads: int = 1):
    """Incremental verification of the target rows [r0, r1).  `out` carries accept_len, token,
    p_draft, resid_mass from earlier calls (decided sequences and untested positions keep their
    values); returns the updated dict with state [B] i32 and borderline_count of this call."""
    l = _f32(target_logits)
    B, G1, V = _rows(l)
    G = G1 - 1
    T = _f32(temperature)
    gm = None if gamma is None else _i32(gamma)
    st = None if state_in is None else _i32(state_in)
    tok_in = _i32(draft_tok).reshape(B, G)
    qi = _i32(q_idx)
    qp = _f32(q_prob)
    qc = _i32(q_count).reshape(B, G)
    k_max = qi.shape[-1] if qi.ndim == 3 and G > 0 else 1
    ua = _f32(u_accept).reshape(B, G)
    ur = _f32(u_resample)
    assert ur.shape == (B, 2)
    if out is None:
        out = {"accept_len": np.full((B,), -2, np.int32), "token": np.full((B,), -2, np.int32),
               "p_draft": np.full((B, G), np.nan, np.float64), "resid_mass": np.full((B, G), np.nan, np.float64)}
    out = {k: np.ascontiguousarray(v).copy() for k, v in out.items() if k in ("accept_len", "token", "p_draft", "resid_mass")}
    border = np.zeros((B,), np.int64)
    state = np.empty((B,), np.int32)
    rc = _load().pso_verify_range(_p(l), ctypes.c_long(B), ctypes.c_long(G), ctypes.c_long(V), ctypes.c_long(V),
                                  _p(T), _p(gm), ctypes.c_long(r0), ctypes.c_long(r1), _p(st), _p(tok_in), _p(qi),
                                  _p(qp), _p(qc), ctypes.c_int(k_max), _p(ua), _p(out["accept_len"]),
                                  _p(out["p_draft"]), _p(out["resid_mass"]), _p(border), _p(ur), _p(out["token"]),
                                  _p(state), ctypes.c_long(chunk), ctypes.c_int(nthreads))
    if rc != 0:
        raise ValueError(f"pso_verify_range failed: {rc}")
    out["state"] = state
    out["borderline_count"] = int(border.sum())
    return out


def residual_sample(target_logits, temperature, pos, q_idx, q_prob, q_count, u_resample,
                    chunk: int = CHUNK, nthreads: int = 1):
    """One token per sequence from row pos[b]: residual against q~ (pos < G, non-empty sparse
    row) or p itself.  Returns (token [B] i32, mass [B] f64)."""
    l = _f32(target_logits)
    B, G1, V = _rows(l)
    G = G1 - 1
    T = _f32(temperature)
    ps = _i32(pos)
    qi = _i32(q_idx)
    qp = _f32(q_prob)
    qc = _i32(q_count)
    k_max = qi.shape[-1] if G > 0 else 1
    ur = _f32(u_resample)
    assert ur.shape == (B, 2) and ps.shape == (B,)
    token = np.empty((B,), np.int32)
    mass = np.empty((B,), np.float64)
    rc = _load().pso_residual_sample(_p(l), ctypes.c_long(B), ctypes.c_long(G), ctypes.c_long(V),
                                     ctypes.c_long(V), _p(T), _p(ps), _p(qi), _p(qp), _p(qc),
                                     ctypes.c_int(k_max), _p(ur), _p(token), _p(mass),
                                     ctypes.c_long(chunk), ctypes.c_int(nthreads))
    if rc != 0:
        raise ValueError(f"pso_residual_sample failed: {rc}")
    return token, mass


def target_topk(target_logits, temperature, pos, k: int, nthreads: int = 1):
    """The paper's downlink payload (Eq. 4): target_logits fp32 [B, R, V], row pos[b] of each
    sequence -> (p_idx [B,k] i32, p_prob [B,k] f32 raw probabilities, p_count [B] i32)."""
    l = _f32(target_logits)
    B, R, V = _rows(l)
    T = _f32(temperature)
    ps = _i32(pos)
    assert T.shape == (B,) and ps.shape == (B,)
    p_idx = np.empty((B, k), np.int32)
    p_prob = np.empty((B, k), np.float32)
    p_count = np.empty((B,), np.int32)
    rc = _load().pso_target_topk(_p(l), ctypes.c_long(B), ctypes.c_long(R), ctypes.c_long(V), ctypes.c_long(V),
                                 _p(T), _p(ps), ctypes.c_int(k), _p(p_idx), _p(p_prob), _p(p_count),
                                 ctypes.c_int(nthreads))
    if rc != 0:
        raise ValueError(f"pso_target_topk failed: {rc}")
    return p_idx, p_prob, p_count


def edge_resample(draft_logits, temperature, pos, p_idx, p_prob, p_count, u, nthreads: int = 1):
    """The paper's edge-side correction: draft_logits fp32 [B, R, V] (the drafter's own rows), row
    pos[b]; the transmitted components (p_idx, p_prob, p_count); one uniform per sequence ->
    (token [B] i32, mass [B] f64)."""
    l = _f32(draft_logits)
    B, R, V = _rows(l)
    T = _f32(temperature)
    ps = _i32(pos)
    pi = _i32(p_idx)
    pp = _f32(p_prob)
    pc = _i32(p_count)
    uu = _f32(u)
    k = pi.shape[-1]
    assert pi.shape == (B, k) and pp.shape == (B, k) and pc.shape == (B,) and uu.shape == (B,) and ps.shape == (B,)
    token = np.empty((B,), np.int32)
    mass = np.empty((B,), np.float64)
    rc = _load().pso_edge_resample(_p(l), ctypes.c_long(B), ctypes.c_long(R), ctypes.c_long(V), ctypes.c_long(V),
                                   _p(T), _p(ps), _p(pi), _p(pp), _p(pc), ctypes.c_int(k), _p(uu), _p(token),
                                   _p(mass), ctypes.c_int(nthreads))
    if rc != 0:
        raise ValueError(f"pso_edge_resample failed: {rc}")
    return token, mass
