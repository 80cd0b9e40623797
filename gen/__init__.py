"""Seeded synthetic inputs for the separate-rejection-sampling hot path.

This module only produces *inputs* (logits, temperatures, uniforms, truncation
parameters).  It holds none of the method's arithmetic: no softmax, no top-k,
no accept test, no sampling.  Both the CPU oracle and the CUDA path consume the
bits produced here; neither of them is imported from here.

The logits have a heavy Zipf-like tail (Sec. 3.3 of the paper observes that
language-model distributions do) and stand in for the Llama-3 (V = 128 256) and
Qwen3 (V = 151 936) vocabularies the paper evaluates on (Sec. 3.3, Sec. 4.1).
For every (sequence b, position i in [0, gamma]):

    rank   = a seeded uniformly random permutation of 1..V
    base_v = -s * ln(rank_v) + sigma_d * N(0, 1)
    draft  = base                       (positions i < gamma only)
    target = c * base + sigma_t * N(0, 1)

generated in fp32 and rounded once (round-to-nearest-even) to the workload's
storage type.  Uniforms are fp32 in [0, 1).
"""
from __future__ import annotations

import dataclasses
from typing import Dict, Optional

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    """One synthetic workload: shapes, logit recipe and truncation parameters."""

    name: str
    V: int
    B: int
    G: int                      # gamma: draft tokens per sequence (+1 bonus target row)
    dtype: str                  # "f32" | "bf16": storage type of the logits
    s: float                    # Zipf exponent
    sigma_d: float              # std of the noise added to the draft logits
    corr: Optional[float]       # target = corr * base + sigma_t * N; None -> per-sequence rho
    sigma_t: float
    T: Optional[float]          # temperature; None -> per-sequence U(0.5, 1.2)
    top_k: int                  # 0 = off
    top_p: float                # >= 1 = off
    k_max: int                  # capacity of a sparse row

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def bytes_per_logit(self) -> int:
        return 4 if self.dtype == "f32" else 2


# The five configurations of the benchmark definition (1-based numbering).
WORKLOADS: Dict[str, Workload] = {
    "config1": Workload("config1", V=32000, B=1, G=4, dtype="f32", s=1.1, sigma_d=1.5,
                        corr=0.8, sigma_t=1.0, T=1.0, top_k=32, top_p=1.0, k_max=32),
    "config2": Workload("config2", V=128256, B=8, G=5, dtype="bf16", s=1.2, sigma_d=1.5,
                        corr=0.85, sigma_t=0.8, T=0.8, top_k=0, top_p=0.95, k_max=64),
    "config3": Workload("config3", V=151936, B=64, G=8, dtype="bf16", s=1.0, sigma_d=1.5,
                        corr=0.7, sigma_t=1.2, T=0.7, top_k=128, top_p=1.0, k_max=128),
    # per-sequence correlation rho ~ U(0.5, 0.95): target = rho*base + sqrt(1-rho^2)*1.5*N;
    # per-sequence temperature ~ U(0.5, 1.2)
    "config4": Workload("config4", V=128256, B=256, G=6, dtype="bf16", s=1.1, sigma_d=1.5,
                        corr=None, sigma_t=1.5, T=None, top_k=0, top_p=0.9, k_max=256),
}

SWEEP_V = (32000, 128256, 151936, 262144)
SWEEP_K = (8, 64, 512, 1024)


def sweep_workload(V: int, k: int, B: int = 512) -> Workload:
    """One point of the bandwidth sweep (configuration 5)."""
    return Workload(f"config5_V{V}_k{k}", V=V, B=B, G=8, dtype="bf16", s=1.1, sigma_d=1.5,
                    corr=0.8, sigma_t=1.0, T=1.0, top_k=k, top_p=1.0, k_max=k)


def scaled(w: Workload, **changes) -> Workload:
    """A copy of a workload with some fields replaced (smaller B or V for tests)."""
    return dataclasses.replace(w, **changes)


def _seq_block(w: Workload) -> int:
    # bound temporaries to roughly 2^26 elements per block of sequences
    per_seq = (w.G + 1) * w.V
    return max(1, min(w.B, (1 << 26) // per_seq))


def make_inputs(w: Workload, seed: int, device: str | torch.device = "cpu") -> Dict[str, torch.Tensor]:
    """Generate one batch of inputs for a workload.

    Returns a dict of tensors on ``device``:
      draft_logits  [B, G, V]    storage dtype
      target_logits [B, G+1, V]  storage dtype
      temperature   [B]          fp32
      u_draft       [B, G]       fp32 in [0, 1)
      u_accept      [B, G]       fp32 in [0, 1)
      u_resample    [B, 2]       fp32 in [0, 1)

    The stream of random numbers depends on the device type (torch's CPU and
    CUDA generators differ), so a test generates once and copies the bits to
    the other side.
    """
    device = torch.device(device)
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    B, G, V = w.B, w.G, w.V
    dt = w.torch_dtype

    draft = torch.empty((B, G, V), dtype=dt, device=device)
    target = torch.empty((B, G + 1, V), dtype=dt, device=device)

    if w.T is None:
        temperature = 0.5 + 0.7 * torch.rand((B,), generator=g, device=device, dtype=torch.float32)
    else:
        temperature = torch.full((B,), float(w.T), dtype=torch.float32, device=device)
    if w.corr is None:
        rho = 0.5 + 0.45 * torch.rand((B,), generator=g, device=device, dtype=torch.float32)
        c_b = rho
        st_b = torch.sqrt(1.0 - rho * rho) * float(w.sigma_t)
    else:
        c_b = torch.full((B,), float(w.corr), dtype=torch.float32, device=device)
        st_b = torch.full((B,), float(w.sigma_t), dtype=torch.float32, device=device)

    blk = _seq_block(w)
    for b0 in range(0, B, blk):
        b1 = min(B, b0 + blk)
        nb = b1 - b0
        keys = torch.rand((nb, G + 1, V), generator=g, device=device, dtype=torch.float32)
        order = torch.argsort(keys, dim=-1)          # a uniformly random permutation per row
        del keys
        rank = torch.empty_like(order)
        ar = torch.arange(1, V + 1, device=device, dtype=order.dtype).expand(nb, G + 1, V)
        rank.scatter_(-1, order, ar)                 # rank[order[j]] = j + 1
        del order, ar
        base = -float(w.s) * torch.log(rank.to(torch.float32))
        del rank
        base += float(w.sigma_d) * torch.randn((nb, G + 1, V), generator=g, device=device,
                                               dtype=torch.float32)
        draft[b0:b1] = base[:, :G, :].to(dt)
        noise = torch.randn((nb, G + 1, V), generator=g, device=device, dtype=torch.float32)
        tgt = c_b[b0:b1, None, None] * base + st_b[b0:b1, None, None] * noise
        target[b0:b1] = tgt.to(dt)
        del base, noise, tgt

    def _uniform(shape):
        u = torch.rand(shape, generator=g, device=device, dtype=torch.float32)
        # torch.rand is in [0, 1) already; clamp guards the fp32 rounding edge
        return u.clamp_(max=1.0 - 2.0 ** -24)   # largest fp32 below 1

    return {
        "draft_logits": draft,
        "target_logits": target,
        "temperature": temperature,
        "u_draft": _uniform((B, G)),
        "u_accept": _uniform((B, G)),
        "u_resample": _uniform((B, 2)),
    }
