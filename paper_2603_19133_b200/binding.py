"""Thin ctypes binding of the picospec C-ABI (include/picospec.h).

Argument marshalling only: every step of the path runs in the CUDA kernels of
libpicospec.so.  torch supplies device memory and the current stream.  There is no CPU
fallback: a missing library or a non-CUDA tensor raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

from . import buildlib as _build

F32, BF16 = 0, 1
OK, EINVAL, ECUDA, ECAPACITY, EDATA = 0, -1, -2, -3, -4
CHUNK = 1024

_lib = None


def lib() -> ctypes.CDLL:
    """Load libpicospec.so (built in-tree by build.build()); fail loudly if it is absent."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if not os.path.exists(path):
            path = _build.build()
        L = ctypes.CDLL(path)
        c_int, c_ll, c_f, vp = ctypes.c_int, ctypes.c_longlong, ctypes.c_float, ctypes.c_void_p
        L.picospec_create.argtypes = [ctypes.POINTER(vp), c_int, c_int, c_int, c_int, c_int]
        L.picospec_destroy.argtypes = [vp]
        L.picospec_strerror.argtypes = [c_int]
        L.picospec_strerror.restype = ctypes.c_char_p
        L.picospec_last_cuda_error.argtypes = [vp]
        L.picospec_status.argtypes = [vp, ctypes.POINTER(c_int), ctypes.POINTER(c_ll), c_int, vp]
        L.picospec_compress.argtypes = [vp, vp, c_int, c_int, c_int, c_int, c_ll, vp, c_int, c_f, c_int,
                                        vp, vp, vp, vp, vp, vp]
        L.picospec_verify.argtypes = [vp, vp, c_int, c_int, c_int, c_int, c_ll, vp, vp, vp, vp, vp, c_int,
                                      vp, vp, vp, vp, vp, vp, vp, vp]
        L.picospec_residual_sample.argtypes = [vp, vp, c_int, c_int, c_int, c_int, c_ll, vp, vp, vp, vp, vp,
                                               c_int, vp, vp, vp, vp]
        L.picospec_profile_enable.argtypes = [vp, c_int]
        L.picospec_profile_period.argtypes = [vp, c_int]
        L.picospec_profile_period.restype = c_int
        L.picospec_profile_read.argtypes = [vp, c_int, ctypes.POINTER(c_f), ctypes.POINTER(c_int), vp]
        L.picospec_target_topk.argtypes = [vp, vp, c_int, c_int, c_int, c_int, c_ll, vp, vp, c_int, vp, vp, vp, vp]
        L.picospec_target_topk.restype = c_int
        L.picospec_edge_resample.argtypes = [vp, vp, c_int, c_int, c_int, c_int, c_ll, vp, vp, vp, vp, vp, c_int,
                                             vp, vp, vp, vp]
        L.picospec_edge_resample.restype = c_int
        L.picospec_verify_range.argtypes = [vp, vp, c_int, c_int, c_int, c_int, c_ll, vp, vp, c_int, c_int, vp, vp,
                                            vp, vp, vp, c_int, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.picospec_verify_range.restype = c_int
        L.picospec_wire_bytes.argtypes = [c_int, c_ll, c_int]
        L.picospec_wire_bytes.restype = c_ll
        L.picospec_wire_pack.argtypes = [vp, vp, vp, vp, c_int, c_int, c_int, vp, c_ll, vp, vp]
        L.picospec_wire_pack.restype = c_int
        L.picospec_wire_unpack.argtypes = [vp, vp, c_ll, c_int, c_int, vp, vp, vp, vp]
        L.picospec_wire_unpack.restype = c_int
        L.picospec_profile_samples.argtypes = [vp, c_int, ctypes.POINTER(c_f), c_int, ctypes.POINTER(c_int), vp]
        L.picospec_profile_samples.restype = c_int
        # vocabulary-parallel verification (driven by vocab_parallel.py)
        L.picospec_vp_local.argtypes = [vp, vp, c_int, c_int, c_int, c_int, c_int, c_ll, c_int, vp, vp, vp, vp, c_int,
                                        vp, vp, vp]
        L.picospec_vp_decide.argtypes = [vp, c_int, c_int, c_int, c_int, c_int, vp, vp, vp, vp, vp, vp, vp, vp, c_int,
                                         vp, vp, vp, vp, vp, vp, vp, vp]
        L.picospec_vp_draw.argtypes = [vp, vp, c_int, c_int, c_int, c_int, c_int, c_ll, c_int, c_int, c_int, vp, vp, vp,
                                       vp, vp, vp, c_int, vp, vp, vp, vp]
        L.picospec_vp_queue.argtypes = [vp, c_int, c_int, vp, vp, vp, vp]
        L.picospec_vp_exact.argtypes = [vp, vp, c_int, c_int, c_int, c_int, c_ll, c_int, vp, vp, vp]
        L.picospec_vp_merge.argtypes = [vp, c_int, vp, vp, vp]
        for f in ("picospec_vp_local", "picospec_vp_decide", "picospec_vp_draw", "picospec_vp_queue",
                  "picospec_vp_exact", "picospec_vp_merge"):
            getattr(L, f).restype = c_int
        L.picospec_wait_limit.argtypes = [vp, ctypes.c_ulonglong]
        L.picospec_wait_limit.restype = c_int
        L.picospec_counters.argtypes = [vp, ctypes.POINTER(c_ll), c_int, vp]
        L.picospec_counters.restype = c_int
        L.picospec_verify_static.argtypes = [vp, c_int, c_int, c_int, c_int, c_ll, vp, vp, vp, vp, vp, c_int,
                                             vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.picospec_verify_static.restype = c_int
        for f in ("picospec_profile_enable", "picospec_profile_read", "picospec_create", "picospec_destroy", "picospec_last_cuda_error", "picospec_status",
                  "picospec_compress", "picospec_verify", "picospec_residual_sample"):
            getattr(L, f).restype = c_int
        _lib = L
    return _lib


class PicospecError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {lib().picospec_strerror(code).decode()} ({code})")


def _check(code: int, what: str):
    if code != OK:
        raise PicospecError(code, what)


def _ptr(t: Optional[torch.Tensor], dtype: Optional[torch.dtype] = None, shape: Optional[Tuple[int, ...]] = None):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("picospec takes CUDA tensors only (there is no CPU path)")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(t.shape)}")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    return ctypes.c_void_p(t.data_ptr())


def _logits(t: torch.Tensor):
    """[B, R, V] logits with a contiguous vocabulary and uniformly pitched rows."""
    if not t.is_cuda or t.dim() != 3 or t.stride(2) != 1:
        raise ValueError("logits must be a CUDA tensor [B, R, V] with contiguous vocabulary")
    B, R, V = t.shape
    pitch = t.stride(1) if R > 1 else (t.stride(0) if B > 1 else V)
    if (R > 1 and B > 1 and t.stride(0) != R * pitch) or pitch < V:
        raise ValueError("rows must be uniformly pitched")
    if t.dtype == torch.float32:
        dt = F32
    elif t.dtype == torch.bfloat16:
        dt = BF16
    else:
        raise ValueError("logits must be float32 or bfloat16")
    return ctypes.c_void_p(t.data_ptr()), dt, B, R, V, pitch


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


STATIC_MAX_ROWS, STATIC_MAX_VOCAB = 256, 262144


def verify_static(target_logits: torch.Tensor, temperature: torch.Tensor, draft_tok: torch.Tensor,
                  q_idx: torch.Tensor, q_prob: torch.Tensor, q_count: torch.Tensor, u_accept: torch.Tensor,
                  u_resample: Optional[torch.Tensor], out: dict):
    """picospec_verify_static: picospec_verify for callers that cannot allocate device memory (an
    engine plugin on a GPU whose memory is already claimed, a loop that must avoid cudaMalloc's
    synchronisation).  It needs no Context; its workspace is a fixed array inside the library, so
    B * (G + 1) <= STATIC_MAX_ROWS and V <= STATIC_MAX_VOCAB.  Nothing is allocated here either:
    every output is a tensor the caller made beforehand and passes in `out`
    (accept_len [B], p_draft [B,G], resid_mass [B,G], borderline_count [1], token [B] or None,
    and optionally device_status [1] int32, slow_rows [1] int64).  Calls on one device share
    the workspace: keep them on one stream.  Returns `out`."""
    p, dt, B, G1, V, pitch = _logits(target_logits)
    G = G1 - 1
    k_max = q_idx.shape[-1]
    _check(lib().picospec_verify_static(
        p, dt, B, G, V, pitch, _ptr(temperature, torch.float32, (B,)),
        _ptr(draft_tok, torch.int32, (B, G)), _ptr(q_idx, torch.int32, (B, G, k_max)),
        _ptr(q_prob, torch.float32, (B, G, k_max)), _ptr(q_count, torch.int32, (B, G)), int(k_max),
        _ptr(u_accept, torch.float32, (B, G)), _ptr(out["accept_len"], torch.int32, (B,)),
        _ptr(out["p_draft"], torch.float32, (B, G)), _ptr(out["resid_mass"], torch.float32, (B, G)),
        _ptr(out["borderline_count"], torch.int32, (1,)), _ptr(u_resample, torch.float32, (B, 2)),
        _ptr(out.get("token"), torch.int32, (B,)), _ptr(out.get("device_status"), torch.int32, (1,)),
        _ptr(out.get("slow_rows"), torch.int64, (1,)), _stream()), "picospec_verify_static")
    return out


def wire_bytes(rows: int, entries: int, prob_type: int = 0) -> int:
    """picospec_wire_bytes: size of a message of `rows` rows holding `entries` (id, prob) pairs."""
    n = lib().picospec_wire_bytes(int(rows), int(entries), int(prob_type))
    if n < 0:
        raise ValueError("picospec_wire_bytes: bad arguments")
    return int(n)


class Context:
    """Owns the library's workspace on one device.  Calls on one context must be ordered on
    one stream at a time; use one context per stream for concurrent work."""

    def __init__(self, max_batch: int, max_gamma: int, max_vocab: int, max_k: int, device: Optional[int] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("picospec needs a CUDA device")
        self.device = torch.cuda.current_device() if device is None else int(device)
        self._h = ctypes.c_void_p()
        _check(lib().picospec_create(ctypes.byref(self._h), self.device, max_batch, max_gamma, max_vocab, max_k),
               "picospec_create")
        self.max_batch, self.max_gamma, self.max_vocab, self.max_k = max_batch, max_gamma, max_vocab, max_k

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().picospec_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def status(self, clear: bool = False) -> Tuple[int, int]:
        """Synchronise the current stream; return (status word, rows re-evaluated in double)."""
        st, slow = ctypes.c_int(0), ctypes.c_longlong(0)
        rc = lib().picospec_status(self._h, ctypes.byref(st), ctypes.byref(slow), int(clear), _stream())
        if rc not in (OK, EDATA):
            raise PicospecError(rc, "picospec_status")
        return st.value, slow.value

    def counters(self, clear: bool = False) -> Tuple[int, int]:
        """Synchronise the current stream; return (rows re-evaluated in double precision, draft rows
        the staged compress kernel handed to the direct kernel), both cumulative."""
        out = (ctypes.c_longlong * 2)()
        _check(lib().picospec_counters(self._h, out, int(clear), _stream()), "picospec_counters")
        return int(out[0]), int(out[1])

    def wait_limit(self, limit_ns: int):
        """picospec_wait_limit: the first time limit of the staged kernels' waits, for later calls."""
        _check(lib().picospec_wait_limit(self._h, int(limit_ns)), "picospec_wait_limit")

    def profile_enable(self, level: int, every: int = 1):
        """0 = off, 1 = time the two streaming kernels, 2 = time every kernel group; only every
        `every`-th launch of a kind is bracketed (picospec_profile_period)."""
        _check(lib().picospec_profile_period(self._h, int(every)), "picospec_profile_period")
        _check(lib().picospec_profile_enable(self._h, int(level)), "picospec_profile_enable")

    def profile_read(self, kind: int) -> Tuple[float, int]:
        """(summed device ms, launches) recorded for one kernel kind since the last read."""
        ms, n = ctypes.c_float(0), ctypes.c_int(0)
        _check(lib().picospec_profile_read(self._h, int(kind), ctypes.byref(ms), ctypes.byref(n), _stream()),
               "picospec_profile_read")
        return ms.value, n.value

    def profile_samples(self, kind: int, capacity: int = 128):
        """Device ms of each launch recorded for one kernel kind since the last read (newest 128 at most)."""
        buf, n = (ctypes.c_float * capacity)(), ctypes.c_int(0)
        _check(lib().picospec_profile_samples(self._h, int(kind), buf, int(capacity), ctypes.byref(n), _stream()),
               "picospec_profile_samples")
        return [float(buf[i]) for i in range(n.value)]

    # -- half 1 -------------------------------------------------------------------------
    def compress(self, draft_logits: torch.Tensor, temperature: torch.Tensor, top_k: int, top_p: float,
                 k_max: int, u_draft: Optional[torch.Tensor] = None, out=None):
        """picospec_compress.  Returns (q_idx [B,G,k_max] i32, q_prob f32, q_count [B,G] i32,
        draft_tok [B,G] i32 or None)."""
        p, dt, B, G, V, pitch = _logits(draft_logits)
        dev = draft_logits.device
        if out is None:
            q_idx = torch.empty((B, G, k_max), dtype=torch.int32, device=dev)
            q_prob = torch.empty((B, G, k_max), dtype=torch.float32, device=dev)
            q_count = torch.empty((B, G), dtype=torch.int32, device=dev)
            tok = torch.empty((B, G), dtype=torch.int32, device=dev) if u_draft is not None else None
        else:
            q_idx, q_prob, q_count, tok = out
        _check(lib().picospec_compress(
            self._h, p, dt, B, G, V, pitch, _ptr(temperature, torch.float32, (B,)), int(top_k), float(top_p),
            int(k_max), _ptr(q_idx, torch.int32, (B, G, k_max)), _ptr(q_prob, torch.float32, (B, G, k_max)),
            _ptr(q_count, torch.int32, (B, G)), _ptr(u_draft, torch.float32, (B, G)),
            _ptr(tok, torch.int32, (B, G)), _stream()), "picospec_compress")
        return q_idx, q_prob, q_count, tok

    # -- half 2a (+2b fused) ------------------------------------------------------------
    def verify(self, target_logits: torch.Tensor, temperature: torch.Tensor, draft_tok: torch.Tensor,
               q_idx: torch.Tensor, q_prob: torch.Tensor, q_count: torch.Tensor, u_accept: torch.Tensor,
               u_resample: Optional[torch.Tensor] = None, out=None):
        """picospec_verify.  Returns dict(accept_len [B], p_draft [B,G], resid_mass [B,G],
        borderline_count [1], token [B] or None)."""
        p, dt, B, G1, V, pitch = _logits(target_logits)
        G = G1 - 1
        k_max = q_idx.shape[-1]
        dev = target_logits.device
        if out is None:
            out = {
                "accept_len": torch.empty((B,), dtype=torch.int32, device=dev),
                "p_draft": torch.empty((B, G), dtype=torch.float32, device=dev),
                "resid_mass": torch.empty((B, G), dtype=torch.float32, device=dev),
                "borderline_count": torch.empty((1,), dtype=torch.int32, device=dev),
                "token": torch.empty((B,), dtype=torch.int32, device=dev) if u_resample is not None else None,
            }
        _check(lib().picospec_verify(
            self._h, p, dt, B, G, V, pitch, _ptr(temperature, torch.float32, (B,)),
            _ptr(draft_tok, torch.int32, (B, G)), _ptr(q_idx, torch.int32, (B, G, k_max)),
            _ptr(q_prob, torch.float32, (B, G, k_max)), _ptr(q_count, torch.int32, (B, G)), int(k_max),
            _ptr(u_accept, torch.float32, (B, G)), _ptr(out["accept_len"], torch.int32, (B,)),
            _ptr(out["p_draft"], torch.float32, (B, G)), _ptr(out["resid_mass"], torch.float32, (B, G)),
            _ptr(out["borderline_count"], torch.int32, (1,)), _ptr(u_resample, torch.float32, (B, 2)),
            _ptr(out["token"], torch.int32, (B,)), _stream()), "picospec_verify")
        return out

    def verify_range(self, target_logits: torch.Tensor, temperature: torch.Tensor, gamma: Optional[torch.Tensor],
                     r0: int, r1: int, state_in: Optional[torch.Tensor], draft_tok: torch.Tensor,
                     q_idx: torch.Tensor, q_prob: torch.Tensor, q_count: torch.Tensor, u_accept: torch.Tensor,
                     u_resample: Optional[torch.Tensor] = None, out=None):
        """picospec_verify_range on the target rows [r0, r1).  `out` is the dict of an earlier call
        (its arrays are updated in place; state may alias state_in) or None.  Returns dict(accept_len,
        p_draft, resid_mass, borderline_count, token or None, state [B] i32)."""
        p, dt, B, G1, V, pitch = _logits(target_logits)
        G = G1 - 1
        k_max = q_idx.shape[-1]
        dev = target_logits.device
        if out is None:
            out = {
                "accept_len": torch.full((B,), -2, dtype=torch.int32, device=dev),
                "p_draft": torch.full((B, G), float("nan"), dtype=torch.float32, device=dev),
                "resid_mass": torch.full((B, G), float("nan"), dtype=torch.float32, device=dev),
                "borderline_count": torch.empty((1,), dtype=torch.int32, device=dev),
                "token": torch.full((B,), -2, dtype=torch.int32, device=dev) if u_resample is not None else None,
                "state": torch.empty((B,), dtype=torch.int32, device=dev),
            }
        _check(lib().picospec_verify_range(
            self._h, p, dt, B, G, V, pitch, _ptr(temperature, torch.float32, (B,)), _ptr(gamma, torch.int32, (B,)),
            int(r0), int(r1), _ptr(state_in, torch.int32, (B,)),
            _ptr(draft_tok, torch.int32, (B, G)), _ptr(q_idx, torch.int32, (B, G, k_max)),
            _ptr(q_prob, torch.float32, (B, G, k_max)), _ptr(q_count, torch.int32, (B, G)), int(k_max),
            _ptr(u_accept, torch.float32, (B, G)), _ptr(out["accept_len"], torch.int32, (B,)),
            _ptr(out["p_draft"], torch.float32, (B, G)), _ptr(out["resid_mass"], torch.float32, (B, G)),
            _ptr(out["borderline_count"], torch.int32, (1,)), _ptr(u_resample, torch.float32, (B, 2)),
            _ptr(out["token"], torch.int32, (B,)), _ptr(out["state"], torch.int32, (B,)), _stream()),
            "picospec_verify_range")
        return out

    # -- the paper's own data flow (Sec. 3.3) ---------------------------------------------------
    def target_topk(self, target_logits: torch.Tensor, temperature: torch.Tensor, pos: torch.Tensor, k: int,
                    out=None):
        """picospec_target_topk.  Returns (p_idx [B,k] i32, p_prob [B,k] f32 unnormalised, p_count [B] i32);
        `out` = such a triple to write into."""
        p, dt, B, R, V, pitch = _logits(target_logits)
        dev = target_logits.device
        if out is not None:
            p_idx, p_prob, p_count = out
            _ptr(p_idx, torch.int32, (B, k)), _ptr(p_prob, torch.float32, (B, k)), _ptr(p_count, torch.int32, (B,))
        else:
            p_idx = torch.empty((B, k), dtype=torch.int32, device=dev)
            p_prob = torch.empty((B, k), dtype=torch.float32, device=dev)
            p_count = torch.empty((B,), dtype=torch.int32, device=dev)
        _check(lib().picospec_target_topk(
            self._h, p, dt, B, R, V, pitch, _ptr(temperature, torch.float32, (B,)), _ptr(pos, torch.int32, (B,)),
            int(k), _ptr(p_idx), _ptr(p_prob), _ptr(p_count), _stream()), "picospec_target_topk")
        return p_idx, p_prob, p_count

    def edge_resample(self, draft_logits: torch.Tensor, temperature: torch.Tensor, pos: torch.Tensor,
                      p_idx: torch.Tensor, p_prob: torch.Tensor, p_count: torch.Tensor, u: torch.Tensor,
                      want_mass: bool = True, out=None):
        """picospec_edge_resample.  Returns (token [B] i32, mass [B] f32 or None); `out` = such a pair
        to write into."""
        p, dt, B, R, V, pitch = _logits(draft_logits)
        k = p_idx.shape[-1]
        dev = draft_logits.device
        if out is not None:
            token, mass = out
            _ptr(token, torch.int32, (B,)), _ptr(mass, torch.float32, (B,))
        else:
            token = torch.empty((B,), dtype=torch.int32, device=dev)
            mass = torch.empty((B,), dtype=torch.float32, device=dev) if want_mass else None
        _check(lib().picospec_edge_resample(
            self._h, p, dt, B, R, V, pitch, _ptr(temperature, torch.float32, (B,)), _ptr(pos, torch.int32, (B,)),
            _ptr(p_idx, torch.int32, (B, k)), _ptr(p_prob, torch.float32, (B, k)), _ptr(p_count, torch.int32, (B,)),
            int(k), _ptr(u, torch.float32, (B,)), _ptr(token), _ptr(mass), _stream()), "picospec_edge_resample")
        return token, mass

    # -- wire format of the sparse rows (Sec. 3.3) ---------------------------------------------
    def wire_pack(self, q_idx: torch.Tensor, q_prob: torch.Tensor, q_count: torch.Tensor, fp16: bool = False,
                  buf: Optional[torch.Tensor] = None, bytes_out: Optional[torch.Tensor] = None):
        """picospec_wire_pack.  q_idx / q_prob [..., K], q_count [...].  Returns (buf uint8, bytes_out
        int64 [1] on the device: the message is buf[:bytes_out]).  Without `buf` one is allocated for the
        largest message these shapes can give."""
        K = q_idx.shape[-1]
        R = q_count.numel()
        ptype = 1 if fp16 else 0
        if buf is None:
            buf = torch.empty((wire_bytes(R, R * K, ptype),), dtype=torch.uint8, device=q_idx.device)
        if bytes_out is None:
            bytes_out = torch.empty((1,), dtype=torch.int64, device=q_idx.device)
        _check(lib().picospec_wire_pack(
            self._h, _ptr(q_idx, torch.int32), _ptr(q_prob, torch.float32), _ptr(q_count, torch.int32), R, int(K), ptype,
            _ptr(buf, torch.uint8), int(buf.numel()), _ptr(bytes_out, torch.int64, (1,)), _stream()), "picospec_wire_pack")
        return buf, bytes_out

    def wire_unpack(self, buf: torch.Tensor, nbytes: int, rows: int, k: int, out=None):
        """picospec_wire_unpack.  Returns dense (q_idx [rows,k] i32, q_prob [rows,k] f32, q_count [rows] i32)."""
        dev = buf.device
        if out is None:
            out = (torch.empty((rows, k), dtype=torch.int32, device=dev),
                   torch.empty((rows, k), dtype=torch.float32, device=dev),
                   torch.empty((rows,), dtype=torch.int32, device=dev))
        _check(lib().picospec_wire_unpack(
            self._h, _ptr(buf, torch.uint8), int(nbytes), int(rows), int(k), _ptr(out[0], torch.int32, (rows, k)),
            _ptr(out[1], torch.float32, (rows, k)), _ptr(out[2], torch.int32, (rows,)), _stream()), "picospec_wire_unpack")
        return out

    # -- half 2b ---------------------------------------------------------------------
    def residual_sample(self, target_logits: torch.Tensor, temperature: torch.Tensor, pos: torch.Tensor,
                        q_idx: torch.Tensor, q_prob: torch.Tensor, q_count: torch.Tensor,
                        u_resample: torch.Tensor, want_mass: bool = True):
        """picospec_residual_sample.  Returns (token [B] i32, mass [B] f32 or None)."""
        p, dt, B, G1, V, pitch = _logits(target_logits)
        G = G1 - 1
        k_max = q_idx.shape[-1] if G > 0 else 1
        dev = target_logits.device
        token = torch.empty((B,), dtype=torch.int32, device=dev)
        mass = torch.empty((B,), dtype=torch.float32, device=dev) if want_mass else None
        _check(lib().picospec_residual_sample(
            self._h, p, dt, B, G, V, pitch, _ptr(temperature, torch.float32, (B,)), _ptr(pos, torch.int32, (B,)),
            _ptr(q_idx, torch.int32), _ptr(q_prob, torch.float32), _ptr(q_count, torch.int32), int(k_max),
            _ptr(u_resample, torch.float32, (B, 2)), _ptr(token, torch.int32, (B,)),
            _ptr(mass, torch.float32, (B,)), _stream()), "picospec_residual_sample")
        return token, mass
