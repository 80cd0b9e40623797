"""GPU parity for the paper's own data flow (Sec. 3.3): the verifier's Top-K of the target row at
the rejected position (Eq. 4, picospec_target_topk) and the edge's resampling against its dense
row (picospec_edge_resample), against the CPU oracle on the same seeded input bits.  Indices,
counts and tokens must be bit-exact; probabilities and masses agree to 1e-5 relative."""
import numpy as np
import pytest
import torch

import gen
import oracle

pytestmark = pytest.mark.gpu

RTOL = 1e-5


@pytest.fixture(scope="module")
def ps():
    import paper_2603_19133_b200 as ps
    ps.lib()
    return ps


def _np(t):
    return t.detach().float().cpu().numpy() if t.is_floating_point() else t.detach().cpu().numpy()


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _flow(ps, w, k, seed, pos=None):
    """target_topk at pos, then edge_resample, on both sides; returns the pieces."""
    inp = gen.make_inputs(w, seed=seed, device="cuda")
    B, R = w.B, w.G + 1
    tl = inp["target_logits"]
    # the edge's rows: the draft rows plus one more row so that every position has one
    dl = torch.cat([inp["draft_logits"], inp["draft_logits"][:, :1] * 0.5], dim=1).contiguous()
    T = inp["temperature"]
    rng = np.random.default_rng(seed)
    if pos is None:
        pos = rng.integers(0, R, size=B).astype(np.int32)
        pos[0], pos[-1] = 0, R - 1
    u = inp["u_resample"][:, 0].contiguous()
    ctx = ps.Context(B, w.G, w.V, max(k, 1))
    try:
        g_pi, g_pp, g_pc = ctx.target_topk(tl, T, _cuda(pos), k)
        o_pi, o_pp, o_pc = oracle.target_topk(_np(tl), _np(T), pos, k, nthreads=oracle.cores())
        st, _ = ctx.status(clear=True)
        assert np.array_equal(_np(g_pc), o_pc), "p_count"
        assert np.array_equal(_np(g_pi), o_pi), "p_idx"
        np.testing.assert_allclose(_np(g_pp), o_pp, rtol=RTOL, atol=0)
        # both sides resample from the oracle's payload bits
        g_tok, g_mass = ctx.edge_resample(dl, T, _cuda(pos), _cuda(o_pi), _cuda(o_pp), _cuda(o_pc), u)
        o_tok, o_mass = oracle.edge_resample(_np(dl), _np(T), pos, o_pi, o_pp, o_pc, _np(u), nthreads=oracle.cores())
        st2, slow = ctx.status(clear=True)
        assert np.array_equal(_np(g_tok), o_tok), "token"
        ok = o_tok >= 0
        np.testing.assert_allclose(_np(g_mass)[ok], o_mass[ok], rtol=RTOL, atol=1e-12)
        return {"status": st | st2, "slow": slow, "o_tok": o_tok, "o_pc": o_pc}
    finally:
        ctx.close()


@pytest.mark.parametrize("name,B,k", [("config1", 4, 10), ("config2", 8, 10), ("config3", 16, 64), ("config4", 16, 300)])
def test_paper_direction_on_the_benchmark_shapes(ps, name, B, k):
    w = gen.scaled(gen.WORKLOADS[name], B=B)
    r = _flow(ps, w, k, seed=60 + k)
    assert r["status"] == 0 and np.all(r["o_tok"] >= 0)


@pytest.mark.parametrize("V,B,G,k,dtype", [
    (1001, 3, 2, 5, "bf16"),       # unaligned rows: direct kernels
    (4099, 2, 3, 16, "f32"),
    (8200, 3, 1, 1, "bf16"),       # K = 1
    (300, 2, 2, 512, "f32"),       # K >= V: everything transmitted
    (20000, 4, 2, 1024, "bf16"),   # widest payload
])
def test_paper_direction_small_shapes(ps, V, B, G, k, dtype):
    w = gen.Workload("t", V=V, B=B, G=G, dtype=dtype, s=1.1, sigma_d=1.5, corr=0.8, sigma_t=1.0,
                     T=None, top_k=0, top_p=1.0, k_max=k)
    r = _flow(ps, w, k, seed=V + k)
    assert r["status"] == 0


def test_paper_direction_bad_data(ps):
    w = gen.Workload("t", V=9000, B=5, G=2, dtype="bf16", s=1.1, sigma_d=1.5, corr=0.8, sigma_t=1.0,
                     T=1.0, top_k=0, top_p=1.0, k_max=8)
    inp = gen.make_inputs(w, seed=5, device="cuda")
    tl = inp["target_logits"].clone()
    T = inp["temperature"].clone()
    pos = np.array([0, 3, 1, 2, 2], np.int32)          # 3 is outside [0, R)
    tl[2, 1, 77] = float("nan")
    T[3] = 0.0
    ctx = ps.Context(w.B, w.G, w.V, 8)
    try:
        g_pi, g_pp, g_pc = ctx.target_topk(tl, T, _cuda(pos), 8)
        o_pi, o_pp, o_pc = oracle.target_topk(_np(tl), _np(T), pos, 8)
        st, _ = ctx.status(clear=True)
        assert st == (1 | 2 | 4)
        assert np.array_equal(_np(g_pc), o_pc) and list(o_pc) == [8, -1, -1, -1, 8]
        assert np.array_equal(_np(g_pi), o_pi)
        # the edge side: a payload with an index out of range, a count out of range, a NaN row
        dl = inp["target_logits"].clone() * 0.7
        pi, pp, pc = oracle.target_topk(_np(inp["target_logits"]), _np(inp["temperature"]), np.zeros(5, np.int32), 8)
        pi[1, 2] = w.V
        pc[2] = 9
        dl[3, 0, 5] = float("inf")
        u = torch.full((5,), 0.4, device="cuda")
        g_tok, g_mass = ctx.edge_resample(dl, inp["temperature"], _cuda(np.zeros(5, np.int32)), _cuda(pi), _cuda(pp),
                                          _cuda(pc), u)
        o_tok, o_mass = oracle.edge_resample(_np(dl), _np(inp["temperature"]), np.zeros(5, np.int32), pi, pp, pc, _np(u))
        st, _ = ctx.status(clear=True)
        assert st == (2 | 4)
        assert np.array_equal(_np(g_tok), o_tok) and list(o_tok[1:4]) == [-1, -1, -1] and o_tok[0] >= 0
        assert np.all(_np(g_mass)[1:4] == -1)
    finally:
        ctx.close()


def test_edge_resample_near_threshold_uniforms_are_decided_exactly(ps):
    # uniforms within a few fp32 ulps of a boundary of the oracle's cumulative residual: the fp32
    # normaliser cannot decide them, the double-precision pass must, and the tokens must still match
    w = gen.scaled(gen.WORKLOADS["config2"], B=32)
    inp = gen.make_inputs(w, seed=77, device="cuda")
    k = 16
    B, R = w.B, w.G + 1
    pos = (np.arange(B) % R).astype(np.int32)
    tl, T = _np(inp["target_logits"]), _np(inp["temperature"])
    dl = torch.cat([inp["draft_logits"], inp["draft_logits"][:, :1] * 0.5], dim=1).contiguous()
    pi, pp, pc = oracle.target_topk(tl, T, pos, k, nthreads=oracle.cores())
    dln = _np(dl)
    u = np.zeros(B, np.float32)
    rng = np.random.default_rng(3)
    for b in range(B):
        x = dln[b, pos[b]].astype(np.float64) / np.float64(T[b])
        q = np.exp(x - x.max())
        q /= q.sum()
        r = np.maximum(0.0, pp[b].astype(np.float64) - q[pi[b]])
        cum = np.cumsum(r)
        inner = np.nonzero((cum > 0) & (cum < cum[-1]))[0]
        t = inner[len(inner) // 2] if len(inner) else 0
        u[b] = np.float32(cum[t] / cum[-1]) * np.float32(1 + rng.integers(-2, 3) * 6e-8)
    u = np.clip(u, 0, 0.999999).astype(np.float32)
    ctx = ps.Context(B, w.G, w.V, k)
    try:
        g_tok, g_mass = ctx.edge_resample(dl, inp["temperature"], _cuda(pos), _cuda(pi), _cuda(pp), _cuda(pc), _cuda(u))
        o_tok, o_mass = oracle.edge_resample(dln, T, pos, pi, pp, pc, u, nthreads=oracle.cores())
        st, slow = ctx.status(clear=True)
        assert st == 0 and slow > 0
        assert np.array_equal(_np(g_tok), o_tok)
    finally:
        ctx.close()


def test_scalar_uplink_verify_then_downlink_then_edge(ps):
    # the whole exchange of Sec. 3.3 on one GPU: the edge sends the drafted tokens and their scalar
    # q(x); the verifier tests them (one-entry sparse rows), finds the first rejection, extracts the
    # Top-K of its row there; the edge resamples.  Every stage against the oracle.
    w = gen.scaled(gen.WORKLOADS["config3"], B=24)
    inp = gen.make_inputs(w, seed=91, device="cuda")
    B, G, k = w.B, w.G, 32
    T = inp["temperature"]
    ctx = ps.Context(B, G, w.V, k)
    try:
        # the drafter: sample x from its truncated distribution, keep only q(x)
        qi, qp, qc, tok = ctx.compress(inp["draft_logits"], T, k, 1.0, k, inp["u_draft"])
        sel = (qi == tok.unsqueeze(-1))
        qx = (qp * sel).sum(-1)
        s_idx = tok.unsqueeze(-1).contiguous()
        s_prob = qx.unsqueeze(-1).contiguous()
        s_cnt = torch.ones((B, G), dtype=torch.int32, device="cuda")
        ctx.close()
        ctx = ps.Context(B, G, w.V, k)
        g = ctx.verify(inp["target_logits"], T, tok, s_idx, s_prob, s_cnt, inp["u_accept"])
        o = oracle.verify(_np(inp["target_logits"]), _np(T), _np(tok), _np(s_idx), _np(s_prob), _np(s_cnt),
                          _np(inp["u_accept"]), nthreads=oracle.cores())
        assert np.array_equal(_np(g["accept_len"]), o["accept_len"])
        pos = g["accept_len"].clone()
        g_pi, g_pp, g_pc = ctx.target_topk(inp["target_logits"], T, pos, k)
        o_pi, o_pp, o_pc = oracle.target_topk(_np(inp["target_logits"]), _np(T), o["accept_len"], k, nthreads=oracle.cores())
        assert np.array_equal(_np(g_pi), o_pi) and np.array_equal(_np(g_pc), o_pc)
        dl = torch.cat([inp["draft_logits"], inp["draft_logits"][:, :1]], dim=1).contiguous()
        u = inp["u_resample"][:, 1].contiguous()
        g_tok, _ = ctx.edge_resample(dl, T, pos, _cuda(o_pi), _cuda(o_pp), _cuda(o_pc), u)
        o_tok, _ = oracle.edge_resample(_np(dl), _np(T), o["accept_len"], o_pi, o_pp, o_pc, _np(u), nthreads=oracle.cores())
        assert np.array_equal(_np(g_tok), o_tok) and np.all(o_tok >= 0)
        assert ctx.status(clear=True)[0] == 0
    finally:
        ctx.close()
