"""ctypes binding of libviasd.so: argument marshalling only.

Every function mirrors the C entry point of the same name in include/viasd.h; tensors are
torch CUDA tensors whose storage the caller owns (torch is used for device memory and streams,
nothing else).  There is no fallback: if the shared library is missing, importing fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libviasd.so")

VIASD_OK, VIASD_EINVAL, VIASD_ECAPACITY, VIASD_ECUDA, VIASD_EDEVICE, VIASD_EUNSUPPORTED = 0, -1, -2, -3, -4, -5

EXPORTS = ["viasd_workspace_bytes", "viasd_init_model", "viasd_full_forward", "viasd_slim_forward",
           "viasd_tier_accept", "viasd_kv_commit", "viasd_verify_step", "viasd_get_stats",
           "viasd_free_model", "viasd_strerror", "viasd_last_cuda_error", "viasd_gemm_scratch_bytes",
           "viasd_gemm", "viasd_gemm_static", "viasd_kl_cost", "viasd_region_mass", "viasd_launch_count", "viasd_set_timing", "viasd_get_timing",
           "viasd_set_option", "viasd_selftest_wait_expiry", "viasd_gemm_status", "viasd_gemm_static_status",
           "viasd_tier_accept_n", "viasd_kv_commit_slim"]

OPTIONS = {"attention_kernel": 0, "attention_splits": 1, "attention_lo": 2, "accept_team": 3, "dual_max_rows": 4,
           "tk_grid": 5, "tk_flat": 6, "gemm_ring_kb": 7, "gemm_epi_groups": 8}
ATTENTION_KERNELS = {"auto": 0, "mma": 1, "tc": 2, "tk": 3}

TIMING_CLASSES = ["gemm", "attention", "norm", "rope", "embed", "tier_accept", "commit"]


class ViasdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().viasd_strerror(code).decode()
        extra = f" (cuda error {lib().viasd_last_cuda_error()})" if code == VIASD_ECUDA else ""
        super().__init__(f"{where}: {msg} [{code}]{extra}")


class Config(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ff",
                                       "vocab", "dtype")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float),
                ("max_batch", C.c_int), ("max_ctx", C.c_int), ("max_query", C.c_int)]


_PP = C.POINTER(C.c_void_p)


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, _PP) for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2")]


class Cache(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("k_full", "v_full", "k_slim", "v_slim", "len", "pending", "tokens",
                                          "len_full")]


class Draft(C.Structure):
    _fields_ = [("batch", C.c_int), ("n_nodes", C.c_int), ("draft_tok", C.c_void_p), ("parent", C.c_void_p),
                ("prow", C.c_void_p), ("n_prows", C.c_int), ("drafter_logits", C.c_void_p), ("per_sequence", C.c_int)]


class Params(C.Structure):
    _fields_ = [("log_tau_hi", C.c_float), ("log_tau_lo", C.c_float), ("conf_source", C.c_int),
                ("mode", C.c_int), ("temperature", C.c_float), ("alpha", C.c_float), ("beta", C.c_float),
                ("log_acc_rel", C.c_float * 3), ("strict_break", C.c_int), ("emit_bonus", C.c_int),
                ("policy", C.c_int), ("seed", C.c_ulonglong), ("step", C.c_ulonglong)]


class Result(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("tier", "conf", "n_acc", "path", "out_tok", "n_emit", "judge",
                                          "corr_src")]


class Stats(C.Structure):
    _fields_ = [("steps", C.c_ulonglong), ("tier_count", C.c_ulonglong * 3), ("emitted", C.c_ulonglong),
                ("accepted", C.c_ulonglong), ("device_status", C.c_int), ("need_slim", C.c_int),
                ("need_full", C.c_int), ("full_ran", C.c_int), ("full_skipped", C.c_ulonglong)]


class Timing(C.Structure):
    _fields_ = [("ms", C.c_double * 7), ("launches", C.c_longlong * 7), ("dropped", C.c_longlong)]


_lib = None


def lib() -> C.CDLL:
    """Loads libviasd.so; raises if it has not been built (there is no other implementation)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with "
                              "`python -m paper_2606_12243_b200.build` (needs nvcc)")
        l = C.CDLL(LIB_PATH)
        l.viasd_workspace_bytes.restype = C.c_size_t
        l.viasd_workspace_bytes.argtypes = [C.POINTER(Config), C.c_int]
        l.viasd_init_model.argtypes = [C.POINTER(Config), C.POINTER(Weights), C.c_char_p, C.c_void_p, C.c_size_t,
                                       C.POINTER(C.c_void_p)]
        fwd = [C.c_void_p, C.POINTER(Cache), C.POINTER(Draft), C.c_void_p, C.c_void_p]
        l.viasd_full_forward.argtypes = fwd
        l.viasd_slim_forward.argtypes = fwd
        l.viasd_tier_accept.argtypes = [C.c_void_p, C.POINTER(Draft), C.POINTER(Params), C.c_void_p, C.c_void_p,
                                        C.c_int, C.POINTER(Result), C.c_void_p]
        l.viasd_kv_commit.argtypes = [C.c_void_p, C.POINTER(Cache), C.POINTER(Draft), C.POINTER(Result), C.c_void_p]
        l.viasd_kv_commit_slim.argtypes = l.viasd_kv_commit.argtypes
        l.viasd_tier_accept_n.argtypes = [C.c_void_p, C.POINTER(Draft), C.POINTER(Params), C.c_int, C.POINTER(C.c_float),
                                          C.POINTER(C.c_void_p), C.c_int, C.POINTER(Result), C.c_void_p]
        l.viasd_verify_step.argtypes = [C.c_void_p, C.POINTER(Cache), C.POINTER(Draft), C.POINTER(Params),
                                        C.c_void_p, C.c_void_p, C.POINTER(Result), C.c_void_p]
        l.viasd_get_stats.argtypes = [C.c_void_p, C.POINTER(Stats), C.c_void_p]
        l.viasd_free_model.argtypes = [C.c_void_p]
        l.viasd_free_model.restype = None
        l.viasd_strerror.argtypes = [C.c_int]
        l.viasd_strerror.restype = C.c_char_p
        l.viasd_last_cuda_error.restype = C.c_int
        l.viasd_gemm_scratch_bytes.restype = C.c_size_t
        l.viasd_gemm_scratch_bytes.argtypes = [C.c_int, C.c_int, C.c_int]
        l.viasd_gemm.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int,
                                 C.c_void_p, C.c_size_t, C.c_void_p]
        l.viasd_gemm_static.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p]
        l.viasd_kl_cost.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_float, C.c_float, C.c_float, C.c_int,
                                    C.c_float, C.c_void_p, C.c_void_p, C.c_void_p]
        l.viasd_region_mass.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_float, C.c_float, C.c_float,
                                        C.c_void_p, C.c_void_p, C.c_void_p]
        l.viasd_set_option.argtypes = [C.c_void_p, C.c_int, C.c_int]
        l.viasd_gemm_status.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.c_void_p]
        l.viasd_gemm_static_status.argtypes = [C.POINTER(C.c_int), C.c_void_p]
        l.viasd_selftest_wait_expiry.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        l.viasd_launch_count.restype = C.c_ulonglong
        l.viasd_set_timing.argtypes = [C.c_void_p, C.c_int]
        l.viasd_get_timing.argtypes = [C.c_void_p, C.POINTER(Timing), C.c_void_p]
        _lib = l
    return _lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def _check(code: int, where: str) -> None:
    if code != VIASD_OK:
        raise ViasdError(code, where)


def make_config(n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ff, vocab, dtype, max_batch, max_ctx,
                max_query, rms_eps=1e-5, rope_theta=10000.0) -> Config:
    return Config(n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ff, vocab,
                  {"f32": 0, "bf16": 1}.get(dtype, dtype), rms_eps, rope_theta, max_batch, max_ctx, max_query)


def workspace_bytes(cfg: Config, n_routed: int) -> int:
    return int(lib().viasd_workspace_bytes(C.byref(cfg), n_routed))


class Model:
    """Handle returned by init_model; keeps the tensors it borrows alive."""

    def __init__(self, handle: int, cfg: Config, keep):
        self.handle, self.cfg, self._keep = handle, cfg, keep

    def close(self) -> None:
        if self.handle:
            lib().viasd_free_model(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def init_model(cfg: Config, embed: torch.Tensor, lm_head: torch.Tensor, final_norm: torch.Tensor,
               layers: Sequence[dict], route_mask: Sequence[int], workspace: torch.Tensor) -> Model:
    """layers[l] maps "wq".."wd", "norm1", "norm2" to device tensors."""
    L = cfg.n_layers
    assert len(layers) == L and len(route_mask) == L
    arrays = {}
    for name in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2"):
        arrays[name] = (C.c_void_p * L)(*[_ptr(layers[l][name]) for l in range(L)])
    w = Weights(_ptr(embed), _ptr(lm_head), _ptr(final_norm),
                *[C.cast(arrays[n], _PP) for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2")])
    out = C.c_void_p()
    mask = bytes(bytearray(int(bool(z)) for z in route_mask))
    rc = lib().viasd_init_model(C.byref(cfg), C.byref(w), mask, _ptr(workspace),
                                workspace.numel() * workspace.element_size(), C.byref(out))
    _check(rc, "viasd_init_model")
    return Model(out.value, cfg, (embed, lm_head, final_norm, layers, workspace))


def make_cache(k_full, v_full, k_slim, v_slim, length, pending, tokens=None, len_full=None) -> Cache:
    c = Cache(_ptr(k_full), _ptr(v_full), _ptr(k_slim), _ptr(v_slim), _ptr(length), _ptr(pending), _ptr(tokens),
              _ptr(len_full))
    c._keep = (k_full, v_full, k_slim, v_slim, length, pending, tokens, len_full)
    return c


def make_draft(draft_tok, parent, prow, n_prows: int, drafter_logits) -> Draft:
    """parent / prow of shape [N] (one tree for the batch) or [B, N] (a tree per sequence)."""
    B, N = draft_tok.shape
    per_seq = int(parent.dim() == 2)
    assert tuple(parent.shape) == ((B, N) if per_seq else (N,)) and tuple(prow.shape) == tuple(parent.shape)
    d = Draft(B, N, _ptr(draft_tok), _ptr(parent), _ptr(prow), n_prows, _ptr(drafter_logits), per_seq)
    d._keep = (draft_tok, parent, prow, drafter_logits)
    return d


def make_params(log_tau_lo: float, log_tau_hi: float, mode: int = 0, temperature: float = 1.0, alpha: float = 0.0,
                beta: float = 1.0, conf_source: int = 0, log_acc_rel=(0.0, 0.0, 0.0), strict_break: int = 0,
                emit_bonus: int = 0, seed: int = 0, step: int = 0, policy: int = 0) -> Params:
    return Params(log_tau_hi, log_tau_lo, conf_source, mode, temperature, alpha, beta,
                  (C.c_float * 3)(*log_acc_rel), strict_break, emit_bonus, policy, seed, step)


@dataclass
class ResultBuffers:
    tier: torch.Tensor
    conf: torch.Tensor
    n_acc: torch.Tensor
    path: torch.Tensor
    out_tok: torch.Tensor
    n_emit: torch.Tensor
    judge: torch.Tensor
    corr_src: torch.Tensor

    def struct(self) -> Result:
        return Result(*[_ptr(getattr(self, n)) for n in ("tier", "conf", "n_acc", "path", "out_tok", "n_emit",
                                                          "judge", "corr_src")])


def alloc_result(batch: int, n_nodes: int, device="cuda") -> ResultBuffers:
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=device)
    return ResultBuffers(z((batch, n_nodes), torch.uint8), z((batch, n_nodes), torch.float32),
                         z((batch,), torch.int32), z((batch, n_nodes), torch.int32),
                         z((batch, n_nodes + 1), torch.int32), z((batch,), torch.int32),
                         z((batch, n_nodes), torch.uint8), z((batch,), torch.int32))


def full_forward(m: Model, cache: Cache, draft: Draft, logits: torch.Tensor, stream=None) -> None:
    _check(lib().viasd_full_forward(m.handle, C.byref(cache), C.byref(draft), _ptr(logits), _stream(stream)),
           "viasd_full_forward")


def slim_forward(m: Model, cache: Cache, draft: Draft, logits: torch.Tensor, stream=None) -> None:
    _check(lib().viasd_slim_forward(m.handle, C.byref(cache), C.byref(draft), _ptr(logits), _stream(stream)),
           "viasd_slim_forward")


def tier_accept(m: Model, draft: Draft, params: Params, slim_logits, full_logits, phase: int,
                result: ResultBuffers, stream=None) -> None:
    r = result.struct()
    _check(lib().viasd_tier_accept(m.handle, C.byref(draft), C.byref(params), _ptr(slim_logits), _ptr(full_logits),
                                   phase, C.byref(r), _stream(stream)), "viasd_tier_accept")


def tier_accept_n(m: Model, draft: Draft, params: Params, log_tau: Sequence[float], judge_logits: Sequence[torch.Tensor],
                  phase: int, result: ResultBuffers, stream=None) -> None:
    """viasd_tier_accept_n: log_tau descending, judge_logits weakest verifier first and q last (None allowed in phase 1)."""
    n = len(log_tau)
    assert len(judge_logits) == n
    r = result.struct()
    taus = (C.c_float * n)(*[float(t) for t in log_tau])
    ptrs = (C.c_void_p * n)(*[_ptr(t) for t in judge_logits])
    _check(lib().viasd_tier_accept_n(m.handle, C.byref(draft), C.byref(params), n, taus, ptrs, phase, C.byref(r),
                                     _stream(stream)), "viasd_tier_accept_n")


def kv_commit_slim(m: Model, cache: Cache, draft: Draft, result: ResultBuffers, stream=None) -> None:
    r = result.struct()
    _check(lib().viasd_kv_commit_slim(m.handle, C.byref(cache), C.byref(draft), C.byref(r), _stream(stream)),
           "viasd_kv_commit_slim")


def kv_commit(m: Model, cache: Cache, draft: Draft, result: ResultBuffers, stream=None) -> None:
    r = result.struct()
    _check(lib().viasd_kv_commit(m.handle, C.byref(cache), C.byref(draft), C.byref(r), _stream(stream)),
           "viasd_kv_commit")


def verify_step(m: Model, cache: Cache, draft: Draft, params: Params, slim_logits, full_logits,
                result: ResultBuffers, stream=None) -> None:
    r = result.struct()
    _check(lib().viasd_verify_step(m.handle, C.byref(cache), C.byref(draft), C.byref(params), _ptr(slim_logits),
                                   _ptr(full_logits), C.byref(r), _stream(stream)), "viasd_verify_step")


def get_stats(m: Model, stream=None) -> Stats:
    s = Stats()
    _check(lib().viasd_get_stats(m.handle, C.byref(s), _stream(stream)), "viasd_get_stats")
    return s


def gemm_scratch_bytes(rows: int, n: int, k: int) -> int:
    return int(lib().viasd_gemm_scratch_bytes(rows, n, k))


def gemm(x: torch.Tensor, w: torch.Tensor, y: torch.Tensor, scratch: torch.Tensor, stream=None) -> None:
    rows, k = x.shape
    n = w.shape[0]
    dtype = 0 if x.dtype == torch.float32 else 1
    _check(lib().viasd_gemm(_ptr(x), _ptr(w), _ptr(y), rows, n, k, dtype, _ptr(scratch),
                            scratch.numel() * scratch.element_size(), _stream(stream)), "viasd_gemm")


def set_option(m: Model, option: str, value) -> None:
    """viasd_set_option by name; attention_kernel also takes "auto" / "mma" / "tc" / "tk"."""
    if option == "attention_kernel" and isinstance(value, str):
        value = ATTENTION_KERNELS[value]
    _check(lib().viasd_set_option(m.handle, OPTIONS[option], int(value)), "viasd_set_option")


def selftest_wait_expiry(status: torch.Tensor, limit_us: int, waited_cycles: Optional[torch.Tensor] = None,
                         stream=None) -> None:
    """viasd_selftest_wait_expiry: status int32[1], waited_cycles int64[1] or None (device tensors)."""
    assert status.dtype == torch.int32 and (waited_cycles is None or waited_cycles.dtype == torch.int64)
    _check(lib().viasd_selftest_wait_expiry(_ptr(status), int(limit_us), _ptr(waited_cycles), _stream(stream)),
           "viasd_selftest_wait_expiry")


def gemm_status(scratch: torch.Tensor, n: int, stream=None) -> int:
    out = C.c_int(0)
    _check(lib().viasd_gemm_status(_ptr(scratch), n, C.byref(out), _stream(stream)), "viasd_gemm_status")
    return out.value


def gemm_static_status(stream=None) -> int:
    out = C.c_int(0)
    _check(lib().viasd_gemm_static_status(C.byref(out), _stream(stream)), "viasd_gemm_static_status")
    return out.value


def launch_count() -> int:
    return int(lib().viasd_launch_count())


def set_timing(m: Model, on: bool) -> None:
    _check(lib().viasd_set_timing(m.handle, int(on)), "viasd_set_timing")


def get_timing(m: Model, stream=None) -> dict:
    t = Timing()
    _check(lib().viasd_get_timing(m.handle, C.byref(t), _stream(stream)), "viasd_get_timing")
    out = {n: {"ms": t.ms[i], "launches": int(t.launches[i])} for i, n in enumerate(TIMING_CLASSES)}
    out["dropped"] = int(t.dropped)
    return out


def kl_cost(judge_logits: torch.Tensor, proposal_logits: torch.Tensor, alpha: float = 0.0, beta: float = 1.0,
            temperature: float = 1.0, margin: int = 0, tau: float = 1.0, stream=None):
    """viasd_kl_cost: per-row KL-style cost of the judge against the proposal (Eq. 11) and its sum (Eq. 10).

    fp32 [rows, V] device tensors -> (cost_rows [rows], cost_total [1]), both fp32 device tensors.
    """
    assert judge_logits.dtype == torch.float32 and proposal_logits.dtype == torch.float32
    assert judge_logits.is_contiguous() and proposal_logits.is_contiguous() and judge_logits.shape == proposal_logits.shape
    rows, vocab = judge_logits.shape
    out = torch.empty(rows, dtype=torch.float32, device=judge_logits.device)
    total = torch.empty(1, dtype=torch.float32, device=judge_logits.device)
    _check(lib().viasd_kl_cost(_ptr(judge_logits), _ptr(proposal_logits), rows, vocab, temperature, alpha, beta,
                               int(margin), tau, _ptr(out), _ptr(total), _stream(stream)), "viasd_kl_cost")
    return out, total


def region_mass(gate_logits: torch.Tensor, proposal_logits: torch.Tensor, log_tau_hi: float, log_tau_lo: float,
                temperature: float = 1.0, stream=None):
    """viasd_region_mass: mass of the proposal on the gate's regions A, B, C per row (Eq. B.8-B.10) and its mean.

    fp32 [rows, V] device tensors -> (mass [rows, 3], mean [3]), both fp32 device tensors.
    """
    assert gate_logits.dtype == torch.float32 and proposal_logits.dtype == torch.float32
    assert gate_logits.is_contiguous() and proposal_logits.is_contiguous() and gate_logits.shape == proposal_logits.shape
    rows, vocab = gate_logits.shape
    mass = torch.empty((rows, 3), dtype=torch.float32, device=gate_logits.device)
    mean = torch.empty(3, dtype=torch.float32, device=gate_logits.device)
    _check(lib().viasd_region_mass(_ptr(gate_logits), _ptr(proposal_logits), rows, vocab, temperature, log_tau_hi,
                                   log_tau_lo, _ptr(mass), _ptr(mean), _stream(stream)), "viasd_region_mass")
    return mass, mean


def gemm_static(x: torch.Tensor, w: torch.Tensor, y: torch.Tensor, stream=None) -> None:
    """viasd_gemm_static: bf16 x [rows, k], W [n, k] -> fp32 y [rows, n] with the library's built-in scratch.

    For callers that must not allocate (no scratch tensor to pass).  rows <= 16, n <= 262144.  Calls on one
    device share the scratch: do not let two of them overlap on the GPU.
    """
    rows, k = x.shape
    n = w.shape[0]
    assert x.dtype == torch.bfloat16 and w.dtype == torch.bfloat16 and y.dtype == torch.float32
    _check(lib().viasd_gemm_static(_ptr(x), _ptr(w), _ptr(y), rows, n, k, _stream(stream)), "viasd_gemm_static")
