"""picospec_verify_static: the verify entry point for callers that cannot allocate device memory.

Some callers of this library cannot call cudaMalloc: a plugin running inside a serving engine that
has already reserved all of the GPU's memory for its own pools, or a latency-critical loop that
must not take the device-wide synchronisation an allocation implies.  They cannot create a context
either (creating one allocates the workspace).  For them the library keeps a fixed workspace inside
its device image and exposes picospec_verify_static, which takes only the caller's own buffers.

The test calls it through the C-ABI twice in a row (the second call finds the first call's leftovers
in the shared workspace) and checks every output against picospec_verify on the same inputs and
against the CPU oracle: integers bit-exact, probabilities and residual masses to the tolerance of the
parity tests.  It checks the entry point's own claim as well: the amount of free device memory is
the same after a call as before it.  And it checks that a problem larger than the fixed workspace is
rejected.  This file is collected last so that a run stopping at the first failure has already run
every other test; it also passes alone."""
import numpy as np
import pytest
import torch

import gen
import oracle

pytestmark = pytest.mark.gpu

RTOL = 1e-5
ATOL_MASS = 1e-12    # resolution of 1 - sum min(p, q~) in double precision


def _alloc_out(B, G, dev):
    i32, f32 = torch.int32, torch.float32
    return {"accept_len": torch.full((B,), -7, dtype=i32, device=dev),
            "p_draft": torch.full((B, G), -7.0, dtype=f32, device=dev),
            "resid_mass": torch.full((B, G), -7.0, dtype=f32, device=dev),
            "borderline_count": torch.full((1,), -7, dtype=i32, device=dev),
            "token": torch.full((B,), -7, dtype=i32, device=dev),
            "device_status": torch.full((1,), -7, dtype=i32, device=dev),
            "slow_rows": torch.full((1,), -7, dtype=torch.int64, device=dev)}


def _same(a, b):
    for k in ("accept_len", "token", "borderline_count"):
        assert torch.equal(a[k], b[k]), k
    np.testing.assert_allclose(a["p_draft"].cpu().numpy(), b["p_draft"].cpu().numpy(), rtol=RTOL, atol=0)
    np.testing.assert_allclose(a["resid_mass"].cpu().numpy(), b["resid_mass"].cpu().numpy(), rtol=RTOL,
                               atol=ATOL_MASS)


def _np(t):
    return t.detach().float().cpu().numpy() if t.is_floating_point() else t.detach().cpu().numpy()


def _same_as_oracle(out, inp, tok, qi, qp, qc):
    o = oracle.verify(_np(inp["target_logits"]), _np(inp["temperature"]), _np(tok), _np(qi), _np(qp), _np(qc),
                      _np(inp["u_accept"]), _np(inp["u_resample"]), nthreads=oracle.cores())
    assert np.array_equal(_np(out["accept_len"]), o["accept_len"])
    assert np.array_equal(_np(out["token"]), o["token"])
    assert int(out["borderline_count"].item()) == o["borderline_count"]
    np.testing.assert_allclose(_np(out["p_draft"]), o["p_draft"], rtol=RTOL, atol=0)
    np.testing.assert_allclose(_np(out["resid_mass"]), o["resid_mass"], rtol=RTOL, atol=ATOL_MASS)


@pytest.mark.parametrize("name,B", [("config2", 8), ("config3", 28), ("config1", 1)])
def test_verify_static_matches_verify_on_two_calls_in_a_row(name, B):
    import paper_2603_19133_b200 as ps
    ps.lib()
    w = gen.scaled(gen.WORKLOADS[name], B=B)
    assert w.B * (w.G + 1) <= ps.STATIC_MAX_ROWS and w.V <= ps.STATIC_MAX_VOCAB
    dev = torch.device("cuda")
    ctx = ps.Context(w.B, w.G, w.V, w.k_max)
    try:
        for call, seed in enumerate((911, 912)):
            inp = gen.make_inputs(w, seed=seed, device="cuda")
            qi, qp, qc, tok = ctx.compress(inp["draft_logits"], inp["temperature"], w.top_k, w.top_p, w.k_max,
                                           inp["u_draft"])
            ctx.status(clear=True)                    # count only the verify call's rows below
            ref = ctx.verify(inp["target_logits"], inp["temperature"], tok, qi, qp, qc, inp["u_accept"],
                             inp["u_resample"])
            st, slow = ctx.status(clear=True)
            assert st == 0
            out = _alloc_out(w.B, w.G, dev)           # the caller's buffers, made before the call
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            ps.verify_static(inp["target_logits"], inp["temperature"], tok, qi, qp, qc, inp["u_accept"],
                             inp["u_resample"], out)
            torch.cuda.synchronize()
            # nothing was allocated, by the library or through torch (on the first call of a process the
            # driver may still load the kernels' code, so the claim is checked from the second call on)
            if call > 0:
                assert torch.cuda.mem_get_info()[0] == free_before
            _same(out, ref)
            _same_as_oracle(out, inp, tok, qi, qp, qc)
            assert int(out["device_status"].item()) == 0, f"call {call}"
            assert int(out["slow_rows"].item()) == slow, f"call {call}"
    finally:
        ctx.close()


def test_verify_static_reports_bad_data_per_call():
    import paper_2603_19133_b200 as ps
    w = gen.scaled(gen.WORKLOADS["config2"], B=4)
    dev = torch.device("cuda")
    inp = gen.make_inputs(w, seed=77, device="cuda")
    ctx = ps.Context(w.B, w.G, w.V, w.k_max)
    try:
        qi, qp, qc, tok = ctx.compress(inp["draft_logits"], inp["temperature"], w.top_k, w.top_p, w.k_max,
                                       inp["u_draft"])
        bad_T = inp["temperature"].clone()
        bad_T[2] = 0.0
        out = _alloc_out(w.B, w.G, dev)
        ps.verify_static(inp["target_logits"], bad_T, tok, qi, qp, qc, inp["u_accept"], inp["u_resample"], out)
        torch.cuda.synchronize()
        assert int(out["device_status"].item()) == 1          # temperature bit
        assert int(out["accept_len"][2].item()) == -1 and int(out["token"][2].item()) == -1
        # the status word is per call: a clean call right after reads zero
        out2 = _alloc_out(w.B, w.G, dev)
        ps.verify_static(inp["target_logits"], inp["temperature"], tok, qi, qp, qc, inp["u_accept"],
                         inp["u_resample"], out2)
        torch.cuda.synchronize()
        assert int(out2["device_status"].item()) == 0
        assert bool((out2["accept_len"] >= 0).all())
    finally:
        ctx.close()


def test_verify_static_rejects_what_does_not_fit():
    import paper_2603_19133_b200 as ps
    dev = torch.device("cuda")
    B, G, V, K = 64, 4, 2048, 8          # 320 rows > STATIC_MAX_ROWS
    i32, f32 = torch.int32, torch.float32
    tl = torch.zeros((B, G + 1, V), dtype=f32, device=dev)
    T = torch.ones((B,), dtype=f32, device=dev)
    tok = torch.zeros((B, G), dtype=i32, device=dev)
    qi = torch.zeros((B, G, K), dtype=i32, device=dev)
    qp = torch.zeros((B, G, K), dtype=f32, device=dev)
    qc = torch.ones((B, G), dtype=i32, device=dev)
    u = torch.zeros((B, G), dtype=f32, device=dev)
    ur = torch.zeros((B, 2), dtype=f32, device=dev)
    with pytest.raises(ps.PicospecError) as e:
        ps.verify_static(tl, T, tok, qi, qp, qc, u, ur, _alloc_out(B, G, dev))
    assert e.value.code == ps.binding.ECAPACITY
    # a vocabulary beyond the fixed workspace is rejected the same way
    B, V = 1, ps.STATIC_MAX_VOCAB + 1024
    tl = torch.zeros((B, G + 1, V), dtype=torch.bfloat16, device=dev)
    with pytest.raises(ps.PicospecError) as e:
        ps.verify_static(tl, T[:B], tok[:B], qi[:B], qp[:B], qc[:B], u[:B], ur[:B], _alloc_out(B, G, dev))
    assert e.value.code == ps.binding.ECAPACITY
