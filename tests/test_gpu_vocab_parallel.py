"""GPU parity for vocabulary-parallel verification (picospec_vp_*; Sec. 4.1: the verifier spans two to
four GPUs, its logits arrive sharded along the vocabulary).  One GPU is available, so the slices of
all ranks live in one memory, each rank has its own context and buffers, and the two kinds of
exchange between the calls (all-gather, element-wise maximum) are copies; every kernel of the path
runs exactly as it would on separate devices.  The results must equal the CPU oracle on the whole
vocabulary: tokens, accept lengths and the borderline count bit for bit, probabilities and residual
masses to 1e-5."""
import numpy as np
import pytest
import torch

import gen
import oracle

pytestmark = pytest.mark.gpu

RTOL = 1e-5
ATOL_MASS = 1e-12    # resolution of 1 - sum min(p, q~) in double precision


def _np(t):
    return t.detach().float().cpu().numpy() if t.is_floating_point() else t.detach().cpu().numpy()


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _run(w, inp, ranks, u_accept=None, u_resample=None, pad=0):
    import paper_2603_19133_b200 as ps
    from paper_2603_19133_b200 import vocab_parallel as vp
    tl, T = inp["target_logits"], inp["temperature"]
    ua = inp["u_accept"] if u_accept is None else u_accept
    ur = inp["u_resample"] if u_resample is None else u_resample
    o_qi, o_qp, o_qc, o_tok = oracle.compress(_np(inp["draft_logits"]), _np(T), w.top_k, w.top_p, w.k_max,
                                              _np(inp["u_draft"]), nthreads=oracle.cores())
    o = oracle.verify(_np(tl), _np(T), o_tok, o_qi, o_qp, o_qc, _np(ua), _np(ur), nthreads=oracle.cores())
    qi, qp, qc, tok = _cuda(o_qi), _cuda(o_qp), _cuda(o_qc), _cuda(o_tok)
    states, ctxs = [], []
    for r in range(ranks):
        v0, v1 = vp.slice_bounds(w.V, ranks, r)
        if pad:     # rows with a pitch larger than the slice, starting off a 16-byte boundary
            buf = torch.empty((w.B, w.G + 1, v1 - v0 + pad), dtype=tl.dtype, device="cuda")
            sl = buf[:, :, 1:1 + v1 - v0]
            sl.copy_(tl[:, :, v0:v1])
        else:
            sl = tl[:, :, v0:v1].contiguous()
        ctx = ps.Context(w.B, w.G, w.V, w.k_max)
        ctxs.append(ctx)
        states.append(vp.RankState(ctx, r, ranks, w.V, sl))
    try:
        rep = lambda t: [t] * ranks
        outs = vp.verify_sharded(states, vp.LocalExchange(ranks), rep(T), rep(tok), rep(qi), rep(qp), rep(qc), rep(ua),
                                 rep(ur))
        torch.cuda.synchronize()
        status = 0
        slow = 0
        for ctx in ctxs:
            st, sl_rows = ctx.status(clear=True)
            status |= st
            slow = max(slow, sl_rows)
    finally:
        for ctx in ctxs:
            ctx.close()
    ok = o["accept_len"] >= 0
    for g in outs:          # every rank ends with the same results
        assert np.array_equal(_np(g["accept_len"]), o["accept_len"]), "accept_len"
        assert np.array_equal(_np(g["token"]), o["token"]), "token"
        assert int(g["borderline_count"].item()) == o["borderline_count"], "borderline_count"
        np.testing.assert_allclose(_np(g["p_draft"])[ok], o["p_draft"][ok], rtol=RTOL, atol=0)
        np.testing.assert_allclose(_np(g["resid_mass"])[ok], o["resid_mass"][ok], rtol=RTOL, atol=ATOL_MASS)
    return status, slow, o, outs


@pytest.mark.parametrize("name,B,ranks", [("config2", 8, 2), ("config3", 16, 4), ("config4", 24, 3), ("config1", 2, 2)])
def test_sharded_verify_matches_the_oracle(name, B, ranks):
    w = gen.scaled(gen.WORKLOADS[name], B=B)
    inp = gen.make_inputs(w, seed=9100 + ranks, device="cuda")
    status, _, _, _ = _run(w, inp, ranks)
    assert status == 0


def test_sharded_verify_ragged_vocabulary_and_unaligned_rows():
    # a vocabulary that is not a multiple of the chunk (the last rank's last chunk is ragged), slices whose
    # rows start off a 16-byte boundary (the statistics pass then reads them directly), fp32 and bf16
    for dtype, V in (("bf16", 50304 + 77), ("f32", 20000)):
        w = gen.Workload("t", V=V, B=5, G=3, dtype=dtype, s=1.1, sigma_d=1.5, corr=0.8, sigma_t=1.0, T=None,
                         top_k=0, top_p=0.9, k_max=48)
        inp = gen.make_inputs(w, seed=9200, device="cuda")
        for ranks, pad in ((2, 0), (3, 9)):
            status, _, _, _ = _run(w, inp, ranks, pad=pad)
            assert status == 0


def test_sharded_verify_decides_close_calls_in_double_precision():
    # uniforms placed next to the accept threshold and next to a chunk boundary of the sampled row's
    # cumulative distribution: the fast pass must hand these sequences to the double-precision pass, on
    # every rank alike, and the owner of the picked chunk must draw the oracle's token
    w = gen.scaled(gen.WORKLOADS["config2"], B=12)
    inp = gen.make_inputs(w, seed=9300, device="cuda")
    tl, T = _np(inp["target_logits"]), _np(inp["temperature"])
    o_qi, o_qp, o_qc, o_tok = oracle.compress(_np(inp["draft_logits"]), T, w.top_k, w.top_p, w.k_max, _np(inp["u_draft"]))
    ref = oracle.verify(tl, T, o_tok, o_qi, o_qp, o_qc, _np(inp["u_accept"]), _np(inp["u_resample"]))
    ua = _np(inp["u_accept"]).copy()
    ur = _np(inp["u_resample"]).copy()
    for b in range(0, w.B, 2):
        # accept test: u just beside p(x)/q~(x) at the first position
        x = o_tok[b, 0]
        k = int(np.nonzero(o_qi[b, 0, :o_qc[b, 0]] == x)[0][0])
        ratio = ref["p_draft"][b, 0] / np.float64(o_qp[b, 0, k])
        if ratio < 1.0:
            ua[b, 0] = np.float32(ratio * (1.0 + 2e-7))
    for b in range(1, w.B, 2):
        # level 1: u1 on a chunk boundary of the residual's cumulative masses (to fp32 resolution)
        ur[b, 0] = np.float32(0.5)
    status, slow, _, _ = _run(w, inp, 2, u_accept=_cuda(ua), u_resample=_cuda(ur))
    assert status == 0
    assert slow > 0          # some sequence did take the double-precision pass


def test_sharded_verify_reports_bad_data():
    w = gen.scaled(gen.WORKLOADS["config2"], B=6)
    inp = gen.make_inputs(w, seed=9400, device="cuda")
    inp["target_logits"][2, 1, 70000] = float("nan")       # in the second rank's slice
    inp["temperature"][4] = 0.0
    status, _, o, outs = _run(w, inp, 2)
    assert status & 2 and status & 1
    assert o["accept_len"][2] == -1 and o["accept_len"][4] == -1 and o["accept_len"][0] >= 0


def test_argument_checks():
    import paper_2603_19133_b200 as ps
    from paper_2603_19133_b200 import vocab_parallel as vp
    w = gen.scaled(gen.WORKLOADS["config2"], B=2)
    inp = gen.make_inputs(w, seed=1, device="cuda")
    ctx = ps.Context(w.B, w.G, w.V, w.k_max)
    try:
        with pytest.raises(ValueError):
            vp.RankState(ctx, 1, 2, w.V, inp["target_logits"][:, :, :1000].contiguous())      # not this rank's share
        assert vp.chunks_per_rank(128256, 4) == 32 and vp.slice_bounds(128256, 4, 3) == (98304, 128256)
    finally:
        ctx.close()
