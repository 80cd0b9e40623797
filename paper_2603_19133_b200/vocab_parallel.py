"""Vocabulary-parallel verification (picospec_vp_*): marshalling and the exchanges between the calls.

The paper's verifier model runs on two to four GPUs (Sec. 4.1), so its output layer leaves the
target logits sharded along the vocabulary.  Every step of the computation is a kernel of the
library; what lives here is the order of the calls and the two kinds of exchange between them -- an
all-gather and an element-wise maximum over ranks -- done with torch.distributed (NCCL on GPUs;
any backend works, the tensors decide) or, when several ranks' slices live in one process, by
plain copies.
"""
from __future__ import annotations

import ctypes
from typing import List, Optional, Sequence

import torch

from . import binding as _b

CHUNK = _b.CHUNK


# ---- the exchanges ------------------------------------------------------------------------------

class DistExchange:
    """One rank per process: torch.distributed collectives on the tensors' own device."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group
        self.ranks = dist.get_world_size(group)

    def gather(self, locals_: Sequence[torch.Tensor]) -> List[torch.Tensor]:
        (t,) = locals_
        out = torch.empty((self.ranks,) + tuple(t.shape), dtype=t.dtype, device=t.device)
        self.dist.all_gather_into_tensor(out.view(-1), t.contiguous().view(-1), group=self.group)
        return [out]

    def maximum(self, locals_: Sequence[torch.Tensor]) -> List[torch.Tensor]:
        (t,) = locals_
        out = t.clone()
        self.dist.all_reduce(out, op=self.dist.ReduceOp.MAX, group=self.group)
        return [out]


class LocalExchange:
    """All ranks in one process (their slices in one memory): the collectives are copies."""

    def __init__(self, ranks: int):
        self.ranks = ranks

    def gather(self, locals_: Sequence[torch.Tensor]) -> List[torch.Tensor]:
        assert len(locals_) == self.ranks
        out = torch.stack(list(locals_))
        return [out] * self.ranks

    def maximum(self, locals_: Sequence[torch.Tensor]) -> List[torch.Tensor]:
        assert len(locals_) == self.ranks
        out = locals_[0]
        for t in locals_[1:]:
            out = torch.maximum(out, t)
        return [out] * self.ranks


def chunks_per_rank(V: int, ranks: int) -> int:
    """Chunks every rank but the last holds when V is split as evenly as whole chunks allow."""
    nch = (V + CHUNK - 1) // CHUNK
    return (nch + ranks - 1) // ranks


def slice_bounds(V: int, ranks: int, rank: int):
    """Columns [v0, v1) of rank `rank`."""
    per = chunks_per_rank(V, ranks) * CHUNK
    return min(V, rank * per), min(V, (rank + 1) * per)


# ---- one rank's share ---------------------------------------------------------------------------

class RankState:
    """A rank's context, slice and buffers for one verification."""

    def __init__(self, ctx: "_b.Context", rank: int, ranks: int, V: int, slice_logits: torch.Tensor):
        p, dt, B, G1, Vs, pitch = _b._logits(slice_logits)
        self.ctx, self.rank, self.ranks, self.V = ctx, rank, ranks, V
        self.p, self.dt, self.B, self.G, self.Vs, self.pitch = p, dt, B, G1 - 1, Vs, pitch
        self.cpr = chunks_per_rank(V, ranks)
        self.v0 = rank * self.cpr * CHUNK
        if self.v0 + Vs != slice_bounds(V, ranks, rank)[1]:
            raise ValueError("the slice does not match this rank's share of the vocabulary")
        self.slice = slice_logits


def verify_sharded(states: Sequence[RankState], exch, temperature, draft_tok, q_idx, q_prob, q_count, u_accept,
                   u_resample):
    """picospec_vp_*: one verification over the ranks in `states` (one element per rank living in this
    process: one with DistExchange, all of them with LocalExchange).  The small inputs are lists with
    one entry per local rank (replicated data, each on its rank's device).  Returns one dict per local
    rank: accept_len [B], p_draft [B,G], resid_mass [B,G], borderline_count [1], token [B]."""
    L = _b.lib()
    n = len(states)
    st0 = states[0]
    B, G, V, ranks, cpr = st0.B, st0.G, st0.V, st0.ranks, st0.cpr
    k_max = q_idx[0].shape[-1]
    rows = B * (G + 1)
    i32, f32, f64 = torch.int32, torch.float32, torch.float64
    P = _b._ptr

    def stream():
        return _b._stream()

    def dev(i):
        return states[i].slice.device

    # 1. local records and entries
    rec_l = [torch.empty((rows, cpr, 2), dtype=f32, device=dev(i)) for i in range(n)]
    ent_l = [torch.empty((B * G, k_max + 1), dtype=f32, device=dev(i)) for i in range(n)]
    for i, s in enumerate(states):
        with torch.cuda.device(dev(i)):
            _b._check(L.picospec_vp_local(s.ctx._h, s.p, s.dt, B, G, s.Vs, s.v0, s.pitch, cpr,
                                          P(temperature[i], f32, (B,)), P(draft_tok[i], i32, (B, G)),
                                          P(q_idx[i], i32, (B, G, k_max)), P(q_count[i], i32, (B, G)), int(k_max),
                                          P(rec_l[i]), P(ent_l[i]), stream()), "picospec_vp_local")
    rec_a = exch.gather(rec_l)
    ent_a = exch.maximum(ent_l)

    out = [{"accept_len": torch.empty((B,), dtype=i32, device=dev(i)),
            "p_draft": torch.empty((B, G), dtype=f32, device=dev(i)),
            "resid_mass": torch.empty((B, G), dtype=f32, device=dev(i)),
            "borderline_count": torch.empty((1,), dtype=i32, device=dev(i)),
            "token": torch.empty((B,), dtype=i32, device=dev(i))} for i in range(n)]
    pick = [torch.empty((B, 4), dtype=i32, device=dev(i)) for i in range(n)]

    def decide(i, sums):
        s, o = states[i], out[i]
        _b._check(L.picospec_vp_decide(s.ctx._h, B, G, V, ranks, cpr, P(rec_a[i]), P(sums), P(ent_a[i]),
                                       P(temperature[i], f32, (B,)), P(draft_tok[i], i32, (B, G)),
                                       P(q_idx[i], i32, (B, G, k_max)), P(q_prob[i], f32, (B, G, k_max)),
                                       P(q_count[i], i32, (B, G)), int(k_max), P(u_accept[i], f32, (B, G)),
                                       P(u_resample[i], f32, (B, 2)), P(o["accept_len"]), P(o["p_draft"]),
                                       P(o["resid_mass"]), P(o["borderline_count"]), P(pick[i]), stream()),
                  "picospec_vp_decide")

    def draw(i, sums, tf):
        s = states[i]
        _b._check(L.picospec_vp_draw(s.ctx._h, s.p, s.dt, B, G, V, s.v0, s.pitch, s.rank, ranks, cpr, P(rec_a[i]),
                                     P(sums), P(temperature[i], f32, (B,)), P(q_idx[i], i32, (B, G, k_max)),
                                     P(q_prob[i], f32, (B, G, k_max)), P(q_count[i], i32, (B, G)), int(k_max),
                                     P(u_resample[i], f32, (B, 2)), P(pick[i]), P(tf), stream()), "picospec_vp_draw")

    # 2. fast pass: decide, the owners draw, tokens and flags are exchanged, the list is built
    tf_l = [torch.empty((2, B), dtype=i32, device=dev(i)) for i in range(n)]
    for i in range(n):
        with torch.cuda.device(dev(i)):
            decide(i, None)
            draw(i, None, tf_l[i])
    tf_a = exch.maximum(tf_l)
    for i, s in enumerate(states):
        with torch.cuda.device(dev(i)):
            _b._check(L.picospec_vp_queue(s.ctx._h, B, G, P(pick[i]), P(tf_a[i]), P(out[i]["token"]), stream()),
                      "picospec_vp_queue")

    # 3. double-precision pass over the listed sequences (an empty list costs a few empty kernels)
    sum_l = [torch.zeros((rows, cpr), dtype=f64, device=dev(i)) for i in range(n)]
    for i, s in enumerate(states):
        with torch.cuda.device(dev(i)):
            _b._check(L.picospec_vp_exact(s.ctx._h, s.p, s.dt, B, G, s.Vs, s.pitch, cpr, P(temperature[i], f32, (B,)),
                                          P(sum_l[i]), stream()), "picospec_vp_exact")
    sum_a = exch.gather(sum_l)
    tf2_l = [torch.empty((2, B), dtype=i32, device=dev(i)) for i in range(n)]
    for i in range(n):
        with torch.cuda.device(dev(i)):
            decide(i, sum_a[i])
            draw(i, sum_a[i], tf2_l[i])
    tf2_a = exch.maximum(tf2_l)
    for i, s in enumerate(states):
        with torch.cuda.device(dev(i)):
            _b._check(L.picospec_vp_merge(s.ctx._h, B, P(tf2_a[i]), P(out[i]["token"]), stream()), "picospec_vp_merge")
    return out
