"""GPU parity for incremental verification (picospec_verify_range; Sec. 3.2 fast verification,
Sec. 3.3 truncated segments): chains of row ranges with carried state and per-sequence draft
lengths, against the CPU oracle's range routine on the same seeded input bits.  Accept lengths,
tokens, states and the borderline count must be bit-exact; probabilities and residual masses
agree to 1e-5 relative.  Rows outside the range of a call are poisoned on the GPU side to show
that they are never read."""
import numpy as np
import pytest
import torch

import gen
import oracle

pytestmark = pytest.mark.gpu

RTOL = 1e-5
ATOL_MASS = 1e-12    # resolution of 1 - sum min(p, q~) in double precision


@pytest.fixture(scope="module")
def ps():
    import paper_2603_19133_b200 as ps
    ps.lib()
    return ps


def _np(t):
    return t.detach().float().cpu().numpy() if t.is_floating_point() else t.detach().cpu().numpy()


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _case(w, seed):
    inp = gen.make_inputs(w, seed=seed, device="cuda")
    T = inp["temperature"]
    qi, qp, qc, tok = oracle.compress(_np(inp["draft_logits"]), _np(T), w.top_k, w.top_p, w.k_max,
                                      _np(inp["u_draft"]), nthreads=oracle.cores())
    return inp, (qi, qp, qc, tok)


def _chain(ps, w, inp, sparse, cuts, gamma=None, poison=True):
    """Run the same chain of range calls on both sides, comparing after every call."""
    B, G = w.B, w.G
    qi, qp, qc, tok = sparse
    tl, T = inp["target_logits"], inp["temperature"]
    tl_np, T_np = _np(tl), _np(T)
    ua, ur = inp["u_accept"], inp["u_resample"]
    d = dict(qi=_cuda(qi), qp=_cuda(qp), qc=_cuda(qc), tok=_cuda(tok))
    g_gamma = None if gamma is None else _cuda(gamma)
    ctx = ps.Context(B, G, w.V, w.k_max)
    o_out, o_state, g_out, g_state = None, None, None, None
    status = 0
    try:
        for r0, r1 in zip(cuts[:-1], cuts[1:]):
            o_out = oracle.verify_range(tl_np, T_np, gamma, r0, r1, o_state, tok, qi, qp, qc, _np(ua), _np(ur),
                                        out=o_out, nthreads=oracle.cores())
            o_state = o_out["state"]
            seen = tl
            if poison:
                # rows that this call must not read: everything outside [r0, r1)
                seen = tl.clone()
                seen[:, :r0] = float("nan")
                seen[:, r1:] = float("nan")
            g_out = ctx.verify_range(seen, T, g_gamma, r0, r1, g_state, d["tok"], d["qi"], d["qp"], d["qc"], ua, ur,
                                     out=g_out)
            g_state = g_out["state"]
            st, _ = ctx.status(clear=True)
            status |= st
            assert np.array_equal(_np(g_out["state"]), o_out["state"]), f"state after rows [{r0},{r1})"
            assert np.array_equal(_np(g_out["accept_len"]), o_out["accept_len"]), f"accept_len after rows [{r0},{r1})"
            assert np.array_equal(_np(g_out["token"]), o_out["token"]), f"token after rows [{r0},{r1})"
            assert int(g_out["borderline_count"].item()) == o_out["borderline_count"]
            gp, op = _np(g_out["p_draft"]).astype(np.float64), o_out["p_draft"]
            gm, om = _np(g_out["resid_mass"]).astype(np.float64), o_out["resid_mass"]
            assert np.array_equal(np.isnan(gp), np.isnan(op)), "positions tested so far"
            assert np.array_equal(np.isnan(gm), np.isnan(om))
            m = ~np.isnan(op)
            np.testing.assert_allclose(gp[m], op[m], rtol=RTOL, atol=0)
            np.testing.assert_allclose(gm[m], om[m], rtol=RTOL, atol=ATOL_MASS)
    finally:
        ctx.close()
    return o_out, g_out, status


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("cuts", [[0, 7], [0, 1, 2, 3, 4, 5, 6, 7], [0, 3, 7], [0, 2, 5, 6, 7], [0, 6, 7]])
def test_chain_of_ranges(ps, cuts, dtype):
    w = gen.scaled(gen.WORKLOADS["config4"], B=24, dtype=dtype, V=50304)
    inp, sparse = _case(w, seed=6100)
    o, g, st = _chain(ps, w, inp, sparse, cuts)
    assert st == 0
    assert np.all(o["state"] == 0)
    # the chain ends where verifying the whole batch at once ends
    qi, qp, qc, tok = sparse
    full = oracle.verify(_np(inp["target_logits"]), _np(inp["temperature"]), tok, qi, qp, qc, _np(inp["u_accept"]),
                         _np(inp["u_resample"]), nthreads=oracle.cores())
    assert np.array_equal(_np(g["accept_len"]), full["accept_len"])
    assert np.array_equal(_np(g["token"]), full["token"])


def test_whole_range_equals_verify_on_the_gpu(ps):
    # r0 = 0, r1 = G + 1, no gamma, no state: the same kernels must give picospec_verify's outputs bit for bit
    w = gen.scaled(gen.WORKLOADS["config3"], B=16)
    inp, sparse = _case(w, seed=6200)
    qi, qp, qc, tok = (_cuda(x) for x in sparse)
    ctx = ps.Context(w.B, w.G, w.V, w.k_max)
    try:
        a = ctx.verify(inp["target_logits"], inp["temperature"], tok, qi, qp, qc, inp["u_accept"], inp["u_resample"])
        b = ctx.verify_range(inp["target_logits"], inp["temperature"], None, 0, w.G + 1, None, tok, qi, qp, qc,
                             inp["u_accept"], inp["u_resample"])
        for k in ("accept_len", "token", "p_draft", "resid_mass", "borderline_count"):
            assert torch.equal(a[k], b[k]), k
        assert int(b["state"].sum().item()) == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("cuts", [[0, 9], [0, 4, 9], [0, 1, 5, 8, 9]])
def test_truncated_segments(ps, cuts):
    # gamma[b] drafted tokens per sequence, 0 and G included; rows beyond the bonus row are poisoned
    w = gen.scaled(gen.WORKLOADS["config3"], B=20, V=40000)
    inp, sparse = _case(w, seed=6300)
    rng = np.random.default_rng(63)
    gamma = rng.integers(0, w.G + 1, size=w.B).astype(np.int32)
    gamma[0], gamma[1] = 0, w.G
    tl = inp["target_logits"]
    for b in range(w.B):
        tl[b, gamma[b] + 1:] = float("nan")
    # a range call on a sequence whose bonus row lies before r0 is the caller's mistake unless the
    # sequence is already decided; a chain from row 0 decides every sequence at or before row gamma[b]
    o, g, st = _chain(ps, w, inp, sparse, cuts, gamma=gamma, poison=False)
    assert st == 0
    assert np.all(o["state"] == 0)
    qi, qp, qc, tok = sparse
    for b in range(w.B):
        gb = int(gamma[b])
        ref = oracle.verify(_np(tl[b:b + 1, :gb + 1]), _np(inp["temperature"][b:b + 1]), tok[b:b + 1, :gb],
                            qi[b:b + 1, :gb], qp[b:b + 1, :gb], qc[b:b + 1, :gb], _np(inp["u_accept"][b:b + 1, :gb]),
                            _np(inp["u_resample"][b:b + 1]))
        assert int(g["accept_len"][b]) == ref["accept_len"][0] and int(g["token"][b]) == ref["token"][0]


def test_all_accepted_prefix_stays_undecided_then_bonus(ps):
    # the drafter's own rows as the target, and a sparse row that holds the whole (tiny) vocabulary:
    # p = q~ up to rounding, so with u < 1/2 every position is accepted and every call but the last
    # leaves all sequences undecided
    w = gen.Workload("tiny", V=1024, B=6, G=5, dtype="f32", s=1.1, sigma_d=1.0, corr=0.8, sigma_t=1.0, T=1.0,
                     top_k=0, top_p=1.0, k_max=1024)
    inp = gen.make_inputs(w, seed=6400, device="cuda")
    dl = inp["draft_logits"]
    inp["target_logits"] = torch.cat([dl, dl[:, :1]], dim=1).contiguous()
    sparse = oracle.compress(_np(dl), _np(inp["temperature"]), 0, 1.0, w.k_max, _np(inp["u_draft"]))
    inp["u_accept"] = inp["u_accept"] * 0.5
    o, g, st = _chain(ps, w, inp, sparse, [0, 2, 5, 6])
    assert st == 0
    assert np.all(_np(g["accept_len"]) == w.G)


def test_bad_data_inside_and_outside_the_range(ps):
    w = gen.scaled(gen.WORKLOADS["config3"], B=12, V=40000)
    inp, sparse = _case(w, seed=6500)
    qi, qp, qc, tok = sparse
    tl = inp["target_logits"]
    tl[2, 1, 77] = float("nan")        # inside the first range
    tl[3, 6, 77] = float("inf")        # only the second range sees it
    gamma = np.full(w.B, w.G, np.int32)
    gamma[4] = w.G + 1                 # out of range
    gamma[5] = -1
    qc = qc.copy()
    qc[6, 0] = w.k_max + 1             # bad count inside the first range
    o, g, st = _chain(ps, w, inp, (qi, qp, qc, tok), [0, 4, 9], gamma=gamma, poison=False)
    for b in (2, 4, 5, 6):
        assert int(g["accept_len"][b]) == -1 and int(g["token"][b]) == -1
    assert st != 0
    # sequence 3 is wrong only if it got as far as row 6
    assert int(g["accept_len"][3]) == o["accept_len"][3]


def test_argument_checks(ps):
    w = gen.scaled(gen.WORKLOADS["config1"], B=2)
    inp, sparse = _case(w, seed=6600)
    qi, qp, qc, tok = (_cuda(x) for x in sparse)
    ctx = ps.Context(w.B, w.G, w.V, w.k_max)
    try:
        for r0, r1 in [(-1, 2), (2, 2), (3, 1), (0, w.G + 2)]:
            with pytest.raises(Exception):
                ctx.verify_range(inp["target_logits"], inp["temperature"], None, r0, r1, None, tok, qi, qp, qc,
                                 inp["u_accept"], inp["u_resample"])
    finally:
        ctx.close()
