"""GPU parity for the wire codec of the sparse rows (picospec_wire_pack / picospec_wire_unpack;
Sec. 3.3's "(id, prob)" payload): the message bytes must equal the CPU oracle's byte for byte, the
unpacked dense rows must equal the oracle's, and malformed messages are refused as a whole."""
import numpy as np
import pytest
import torch

import gen
import oracle
from oracle import wire

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ps():
    import paper_2603_19133_b200 as ps
    ps.lib()
    return ps


def _np(t):
    return t.detach().cpu().numpy()


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _rows(w, seed):
    inp = gen.make_inputs(w, seed=seed, device="cpu")
    qi, qp, qc, _ = oracle.compress(inp["draft_logits"].float().numpy(), inp["temperature"].numpy(), w.top_k, w.top_p,
                                    w.k_max, inp["u_draft"].numpy(), nthreads=oracle.cores())
    return qi, qp, qc


@pytest.mark.parametrize("fp16", [False, True])
@pytest.mark.parametrize("name,B", [("config1", 1), ("config2", 8), ("config4", 24)])
def test_pack_bytes_and_unpack_rows_match_the_oracle(ps, name, B, fp16):
    w = gen.scaled(gen.WORKLOADS[name], B=B, V=min(gen.WORKLOADS[name].V, 20000))
    qi, qp, qc = _rows(w, 8100 + B)
    R, K = w.B * w.G, w.k_max
    qc = qc.copy()
    if R > 2:
        qc.reshape(-1)[1] = -1                      # an invalid row travels as such
        qi.reshape(R, K)[1] = -1
        qp.reshape(R, K)[1] = 0
    ref = wire.pack(qi, qp, qc, int(fp16))
    ctx = ps.Context(w.B, w.G, w.V, K)
    try:
        buf, nbytes = ctx.wire_pack(_cuda(qi), _cuda(qp), _cuda(qc), fp16=fp16)
        n = int(nbytes.item())
        assert n == ref.size == ps.wire_bytes(R, int(np.maximum(qc, 0).sum()), int(fp16))
        assert np.array_equal(_np(buf[:n]), ref), "message bytes"
        ui, up, uc = ctx.wire_unpack(buf, n, R, K)
        oi, op, oc = wire.unpack(ref, R, K)
        assert np.array_equal(_np(ui), oi) and np.array_equal(_np(uc), oc)
        assert np.array_equal(_np(up), op)          # fp16 -> fp32 is exact on both sides
        if not fp16:
            assert np.array_equal(_np(up), qp.reshape(R, K)) and np.array_equal(_np(ui), qi.reshape(R, K))
        assert ctx.status(clear=True)[0] == 0
    finally:
        ctx.close()


def test_malformed_messages_are_refused_as_a_whole(ps):
    w = gen.scaled(gen.WORKLOADS["config2"], B=4, V=16384)
    qi, qp, qc = _rows(w, 8200)
    R, K = w.B * w.G, w.k_max
    ctx = ps.Context(w.B, w.G, w.V, K)
    try:
        buf, nbytes = ctx.wire_pack(_cuda(qi), _cuda(qp), _cuda(qc))
        n = int(nbytes.item())
        good = buf[:n].clone()

        def refused(b, nb, rows, k):
            ui, up, uc = ctx.wire_unpack(b, nb, rows, k)
            st, _ = ctx.status(clear=True)
            return st == 4 and bool((uc == -1).all()) and bool((ui == -1).all()) and bool((up == 0).all())

        assert refused(good, n, R - 1, K)                      # another number of rows
        assert refused(good, n, R, K - 1)                      # another capacity
        assert refused(good, n - 4, R, K)                      # cut short
        bad = good.clone(); bad[0] ^= 1
        assert refused(bad, n, R, K)                           # wrong magic
        bad = good.clone(); bad[16] = (int(bad[16]) + 1) & 0xFF
        assert refused(bad, n, R, K)                           # counts that do not add up to N
        bad = good.clone(); bad[10] = 2
        assert refused(bad, n, R, K)                           # unknown probability type
        # the oracle refuses the same messages
        for b, nb, rows, k in ((good, n, R - 1, K), (good, n, R, K - 1), (good, n - 4, R, K)):
            assert np.all(wire.unpack(_np(b)[:nb], rows, k)[2] == -1)
        # and the intact message still unpacks
        ui, up, uc = ctx.wire_unpack(good, n, R, K)
        assert np.array_equal(_np(uc), qc.reshape(-1)) and ctx.status(clear=True)[0] == 0
    finally:
        ctx.close()


def test_message_that_does_not_fit_and_bad_counts(ps):
    w = gen.scaled(gen.WORKLOADS["config2"], B=2, V=16384)
    qi, qp, qc = _rows(w, 8300)
    R, K = w.B * w.G, w.k_max
    ctx = ps.Context(w.B, w.G, w.V, K)
    try:
        small = torch.full((64,), 0xAB, dtype=torch.uint8, device="cuda")
        buf, nbytes = ctx.wire_pack(_cuda(qi), _cuda(qp), _cuda(qc), buf=small)
        assert int(nbytes.item()) == -1 and ctx.status(clear=True)[0] == 4
        assert bool((small == 0xAB).all())                      # buf holds no message: nothing was written
        # a buffer that ends inside the counts (16 + 2 R bytes would be needed for them alone), with a
        # guard pattern behind it in the same allocation
        guard = torch.full((256,), 0xCD, dtype=torch.uint8, device="cuda")
        assert 20 < 16 + 2 * R
        buf, nbytes = ctx.wire_pack(_cuda(qi), _cuda(qp), _cuda(qc), buf=guard[:20])
        assert int(nbytes.item()) == -1 and ctx.status(clear=True)[0] == 4
        assert bool((guard == 0xCD).all())
        qc2 = qc.copy().reshape(-1)
        qc2[0] = K + 1                                          # a count beyond the capacity
        buf, nbytes = ctx.wire_pack(_cuda(qi), _cuda(qp), _cuda(qc2))
        n = int(nbytes.item())
        assert ctx.status(clear=True)[0] == 4
        assert np.array_equal(_np(buf[:n]), wire.pack(qi, qp, qc2, 0))      # the row travels as invalid
    finally:
        ctx.close()


def test_full_batch_of_the_benchmark_shape_round_trips(ps):
    # 1536 rows x 256 entries, as picospec_compress leaves them on the device
    w = gen.WORKLOADS["config4"]
    inp = gen.make_inputs(w, seed=8400, device="cuda")
    ctx = ps.Context(w.B, w.G, w.V, w.k_max)
    try:
        qi, qp, qc, _ = ctx.compress(inp["draft_logits"], inp["temperature"], w.top_k, w.top_p, w.k_max, inp["u_draft"])
        for fp16 in (False, True):
            buf, nbytes = ctx.wire_pack(qi, qp, qc, fp16=fp16)
            n = int(nbytes.item())
            assert n == ps.wire_bytes(qc.numel(), int(qc.clamp(min=0).sum().item()), int(fp16))
            ui, up, uc = ctx.wire_unpack(buf, n, qc.numel(), w.k_max)
            assert torch.equal(ui, qi.reshape(-1, w.k_max)) and torch.equal(uc, qc.reshape(-1))
            want = qp.reshape(-1, w.k_max)
            assert torch.equal(up, want.half().float() if fp16 else want)
            ref = wire.pack(_np(qi), _np(qp), _np(qc), int(fp16))
            assert np.array_equal(_np(buf[:n]), ref)
        assert ctx.status(clear=True)[0] == 0
    finally:
        ctx.close()
