"""Thin ctypes binding over ``libespo.so``: same names as the C ABI, argument marshalling only.

Every step of the method runs inside the CUDA library.  PyTorch is used here only to hold
device memory and to name the current stream.  There is no CPU fallback: if the shared
library is missing or no CUDA device is present the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

from . import build as _build

ESPO_OK = 0
ESPO_ERR_NULL, ESPO_ERR_BAD_DTYPE, ESPO_ERR_BAD_SHAPE, ESPO_ERR_ALIGN = -1, -2, -3, -4
ESPO_ERR_CAPACITY, ESPO_ERR_CUDA, ESPO_ERR_BAD_PARAM = -5, -6, -7
ESPO_F32, ESPO_BF16 = 0, 1
ESPO_SAMPLER_FLAT, ESPO_SAMPLER_HIER = 0, 1
ESPO_STOP_ESPO, ESPO_STOP_VALUE_ONLY, ESPO_STOP_REGRET_ONLY, ESPO_STOP_RANDOM = 0, 1, 2, 3
ESPO_ROW_ACTIVE, ESPO_ROW_STOPPED, ESPO_ROW_EOS, ESPO_ROW_TMAX, ESPO_ROW_BAD = 0, 1, 2, 3, 4
ESPO_DEV_BAD_ROW, ESPO_DEV_BAD_SLOT, ESPO_DEV_TIMEOUT, ESPO_DEV_NAN_VALUE, ESPO_DEV_BAD_LENGTHS = 1, 2, 4, 8, 16


class EspoError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().espo_strerror(code).decode()
        if code == ESPO_ERR_CUDA:
            msg += f" [cudaError {lib().espo_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({code})")


class espo_params(C.Structure):
    """Mirror of the C struct: parameters frozen for a rollout batch (Eq. 9-11, Algorithm 1)."""
    _fields_ = [("temperature", C.c_float), ("mu_g", C.c_float), ("sigma2_g", C.c_float),
                ("delta", C.c_float), ("clip_c", C.c_float), ("alpha_s", C.c_float),
                ("beta", C.c_float), ("eps", C.c_float), ("warmup_complete", C.c_int32),
                ("t_max", C.c_int32), ("eos_token", C.c_int32), ("sampler", C.c_int32),
                ("stop_mode", C.c_int32), ("shadow", C.c_int32), ("tau", C.c_float), ("p_random", C.c_float),
                ("want_entropy", C.c_int32), ("top_p", C.c_float), ("top_k", C.c_int32)]


def make_params(temperature=1.0, mu_g=0.0, sigma2_g=1.0, delta=1e-8, clip_c=10.0, alpha_s=0.9, beta=7.0,
                eps=0.2, warmup_complete=1, t_max=8192, eos_token=-1, sampler=ESPO_SAMPLER_HIER,
                stop_mode=ESPO_STOP_ESPO, shadow=0, tau=0.0, p_random=0.0, want_entropy=0, top_p=1.0,
                top_k=0) -> espo_params:
    """Defaults follow the paper's hyper-parameter table (alpha_s 0.9, beta 7.0, eps 0.2, T_max 8192)."""
    return espo_params(temperature, mu_g, sigma2_g, delta, clip_c, alpha_s, beta, eps, warmup_complete, t_max,
                       eos_token, sampler, stop_mode, int(bool(shadow)), tau, p_random, int(bool(want_entropy)), top_p,
                       int(top_k))


_lib = None


def lib():
    """Load ``libespo.so`` (built in-tree).  Raises if it is not there: nothing else can do the work."""
    global _lib
    if _lib is None:
        path = _build.LIB_PATH
        if not os.path.exists(path):
            raise RuntimeError(
                f"{path} is missing: build the CUDA library first (python -m paper_2605_29860_b200.build); "
                "this package has no other implementation to fall back to")
        L = C.CDLL(path)
        vp, i32, i64, u64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_float
        L.espo_init_state.argtypes = [C.POINTER(vp), i32, i32, u64, u64, vp]
        L.espo_reset_state.argtypes = [vp, u64, vp]
        L.espo_free_state.argtypes = [vp]
        L.espo_free_state.restype = None
        L.espo_set_launch_config.argtypes = [vp, i32, i32, i32]
        L.espo_set_dependent_launch.argtypes = [vp, i32]
        L.espo_step.argtypes = [vp, i32, i64, vp, i32, vp, i32, vp, C.POINTER(espo_params), vp, vp, vp]
        L.espo_step_partial.argtypes = [vp, i32, i64, i32, i32, vp, i32, vp, C.POINTER(espo_params), vp, vp]
        L.espo_step_merge.argtypes = [vp, i32, i64, vp, i32, vp, i32, vp, C.POINTER(espo_params), vp, vp, vp]
        L.espo_state_view.argtypes = [vp] + [C.POINTER(vp)] * 11
        L.espo_compact_active.argtypes = [vp, vp, vp, vp]
        L.espo_state_status.argtypes = [vp, C.POINTER(C.c_uint32), vp]
        L.espo_end_batch.argtypes = [vp, f32, f32, f32, f32, f32, i32, C.POINTER(espo_params), C.POINTER(C.c_double), vp]
        L.espo_end_batch_merge.argtypes = [C.POINTER(C.c_double), i32, f32, f32, f32, f32, f32, i32, C.POINTER(espo_params), C.POINTER(C.c_double)]
        L.espo_advantages.argtypes = [vp, vp, vp, vp, i32, i64, f32, f32, f32, vp, vp]
        L.espo_advantages_returns.argtypes = [vp, vp, vp, vp, i32, i64, f32, f32, f32, vp, vp, vp]
        L.espo_advantages_stats.argtypes = [vp, vp, vp, vp, i32, i64, f32, f32, f32, vp, vp, vp, vp]
        L.espo_advantages_padded.argtypes = [vp, vp, vp, vp, i32, i32, f32, f32, f32, vp, vp, vp]
        L.espo_advantages_noalloc.argtypes = [vp, vp, vp, vp, i32, i64, f32, f32, f32, vp, vp, vp]
        L.espo_advantages_reserve.argtypes = [i32, i64]
        L.espo_advantages_status.argtypes = [C.POINTER(C.c_uint32), vp]
        L.espo_strerror.argtypes = [C.c_int]
        L.espo_strerror.restype = C.c_char_p
        L.espo_last_cuda_error.argtypes = []
        for n in ("espo_init_state", "espo_reset_state", "espo_set_launch_config", "espo_step", "espo_step_partial",
                  "espo_step_merge", "espo_state_view",
                  "espo_compact_active", "espo_state_status", "espo_end_batch", "espo_end_batch_merge", "espo_advantages", "espo_advantages_reserve",
                  "espo_advantages_status", "espo_advantages_noalloc", "espo_advantages_returns", "espo_advantages_stats", "espo_advantages_padded",
                  "espo_last_cuda_error"):
            getattr(L, n).restype = C.c_int
        _lib = L
    return _lib


def _check(code: int, where: str) -> None:
    if code != ESPO_OK:
        raise EspoError(code, where)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _dev_ptr(t: Optional[torch.Tensor], name: str) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    return t.data_ptr()


def _dtype_code(t: torch.Tensor, name: str) -> int:
    if t.dtype == torch.float32:
        return ESPO_F32
    if t.dtype == torch.bfloat16:
        return ESPO_BF16
    raise ValueError(f"{name} must be float32 or bfloat16, got {t.dtype}")


class EspoState:
    """Owner of an ``espo_state*``; frees it when collected."""

    def __init__(self, handle: int, capacity: int, V: int, device: torch.device):
        self.handle = C.c_void_p(handle)
        self.capacity = capacity
        self.V = V
        self.device = device

    def close(self) -> None:
        if self.handle:
            lib().espo_free_state(self.handle)
            self.handle = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def espo_init_state(capacity: int, V: int, seed: int, batch_id: int = 0, stream=None) -> EspoState:
    if not torch.cuda.is_available():
        raise RuntimeError("espo_init_state needs a CUDA device; there is no CPU implementation")
    h = C.c_void_p()
    _check(lib().espo_init_state(C.byref(h), capacity, V, seed, batch_id, _stream(stream)), "espo_init_state")
    return EspoState(h.value, capacity, V, torch.device("cuda", torch.cuda.current_device()))


def espo_reset_state(state: EspoState, batch_id: int, stream=None) -> None:
    _check(lib().espo_reset_state(state.handle, batch_id, _stream(stream)), "espo_reset_state")


def espo_free_state(state: EspoState) -> None:
    state.close()


def espo_set_launch_config(state: EspoState, consumer_warps: int = 0, stages: int = 0, ctas_per_sm: int = 0) -> None:
    _check(lib().espo_set_launch_config(state.handle, consumer_warps, stages, ctas_per_sm), "espo_set_launch_config")


def espo_set_dependent_launch(state: EspoState, enable: bool = True) -> None:
    """Let the hierarchical step kernel be set up while the kernel before it in the stream winds down; see ``espo.h``."""
    _check(lib().espo_set_dependent_launch(state.handle, int(bool(enable))), "espo_set_dependent_launch")


def espo_step(logits: torch.Tensor, values: torch.Tensor, state: EspoState, params: espo_params,
              tokens_out: torch.Tensor, stop_out: torch.Tensor, row_ids: Optional[torch.Tensor] = None,
              n_rows: Optional[int] = None, stream=None) -> None:
    """One decode step (Algorithm 1 loop body) for ``logits`` [n_rows, V]; see ``espo.h``."""
    if logits.dim() != 2 or logits.stride(1) != 1:
        raise ValueError("logits must be [n_rows, V] with unit stride along V")
    n = logits.shape[0] if n_rows is None else n_rows
    if logits.shape[1] != state.V:
        raise ValueError(f"logits have V={logits.shape[1]}, state was created for V={state.V}")
    if tokens_out.dtype != torch.int32 or stop_out.dtype != torch.uint8:
        raise ValueError("tokens_out must be int32 and stop_out uint8")
    if row_ids is not None and row_ids.dtype != torch.int32:
        raise ValueError("row_ids must be int32")
    if not values.is_contiguous() or not tokens_out.is_contiguous() or not stop_out.is_contiguous():
        raise ValueError("values, tokens_out and stop_out must be contiguous")
    if min(values.numel(), tokens_out.numel(), stop_out.numel()) < n or (row_ids is not None and row_ids.numel() < n):
        raise ValueError("an argument is shorter than n_rows")
    _check(lib().espo_step(_dev_ptr(logits, "logits"), _dtype_code(logits, "logits"), logits.stride(0),
                           _dev_ptr(values, "values"), _dtype_code(values, "values"),
                           _dev_ptr(row_ids, "row_ids"), n, state.handle, C.byref(params),
                           _dev_ptr(tokens_out, "tokens_out"), _dev_ptr(stop_out, "stop_out"), _stream(stream)),
           "espo_step")


PARTIAL_FLOATS = 8   # an espo_partial is 32 bytes; tensors of partials are float32 [..., 8] (ids and flags bit-cast)


def espo_step_partial(logits_shard: torch.Tensor, vocab_offset: int, state: EspoState, params: espo_params,
                      partial_out: torch.Tensor, row_ids: Optional[torch.Tensor] = None, n_rows: Optional[int] = None,
                      stream=None) -> None:
    """One vocabulary shard's share of a decode step: ``logits_shard`` is [n_rows, v_shard], its first column is
    token ``vocab_offset``; writes one espo_partial per row into ``partial_out`` (float32 [n_rows, 8]); see ``espo.h``."""
    if logits_shard.dim() != 2 or logits_shard.stride(1) != 1:
        raise ValueError("logits_shard must be [n_rows, v_shard] with unit stride along the vocabulary")
    n = logits_shard.shape[0] if n_rows is None else n_rows
    if partial_out.dtype != torch.float32 or not partial_out.is_contiguous() or partial_out.numel() < n * PARTIAL_FLOATS:
        raise ValueError("partial_out must be a contiguous float32 tensor of n_rows * 8 elements")
    if row_ids is not None and (row_ids.dtype != torch.int32 or row_ids.numel() < n):
        raise ValueError("row_ids must be int32 [n_rows]")
    _check(lib().espo_step_partial(_dev_ptr(logits_shard, "logits_shard"), _dtype_code(logits_shard, "logits_shard"),
                                   logits_shard.stride(0), logits_shard.shape[1], vocab_offset,
                                   _dev_ptr(row_ids, "row_ids"), n, state.handle, C.byref(params),
                                   _dev_ptr(partial_out, "partial_out"), _stream(stream)),
           "espo_step_partial")


def espo_step_merge(partials: torch.Tensor, values: torch.Tensor, state: EspoState, params: espo_params,
                    tokens_out: torch.Tensor, stop_out: torch.Tensor, row_ids: Optional[torch.Tensor] = None,
                    n_rows: Optional[int] = None, stream=None) -> None:
    """Merges the shards' partials (float32 [n_shards, rows, 8]) and commits the step like ``espo_step``; see ``espo.h``."""
    if partials.dim() != 3 or partials.shape[2] != PARTIAL_FLOATS or partials.dtype != torch.float32 or \
            not partials.is_contiguous():
        raise ValueError("partials must be a contiguous float32 [n_shards, rows, 8] tensor")
    n = partials.shape[1] if n_rows is None else n_rows
    if tokens_out.dtype != torch.int32 or stop_out.dtype != torch.uint8:
        raise ValueError("tokens_out must be int32 and stop_out uint8")
    if row_ids is not None and row_ids.dtype != torch.int32:
        raise ValueError("row_ids must be int32")
    if not values.is_contiguous() or not tokens_out.is_contiguous() or not stop_out.is_contiguous():
        raise ValueError("values, tokens_out and stop_out must be contiguous")
    if min(values.numel(), tokens_out.numel(), stop_out.numel()) < n or (row_ids is not None and row_ids.numel() < n):
        raise ValueError("an argument is shorter than n_rows")
    _check(lib().espo_step_merge(_dev_ptr(partials, "partials"), partials.shape[0], partials.shape[1],
                                 _dev_ptr(values, "values"), _dtype_code(values, "values"), _dev_ptr(row_ids, "row_ids"),
                                 n, state.handle, C.byref(params), _dev_ptr(tokens_out, "tokens_out"),
                                 _dev_ptr(stop_out, "stop_out"), _stream(stream)),
           "espo_step_merge")


class _DevArray:
    """Minimal __cuda_array_interface__ carrier so torch can view library-owned device memory."""

    def __init__(self, ptr: int, n: int, typestr: str):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": typestr, "data": (ptr, False), "version": 2}


def espo_state_view(state: EspoState) -> dict:
    """Torch views (treat as read-only) of the per-slot arrays: z, g, g_tilde, logp, t, status, t_stop, sum_g, sum_g2."""
    ptrs = [C.c_void_p() for _ in range(11)]
    _check(lib().espo_state_view(state.handle, *[C.byref(p) for p in ptrs]), "espo_state_view")
    names = ["z", "g", "g_tilde", "logp", "t", "status", "t_stop", "sum_g", "sum_g2", "entropy", "sum_h"]
    types = ["<f4", "<f4", "<f4", "<f4", "<i4", "|u1", "<i4", "<f8", "<f8", "<f4", "<f8"]
    with torch.cuda.device(state.device):
        return {n: torch.as_tensor(_DevArray(p.value, state.capacity, ty), device=state.device)
                for n, p, ty in zip(names, ptrs, types)}


def espo_compact_active(state: EspoState, row_ids_out: torch.Tensor, n_active_out: torch.Tensor, stream=None) -> None:
    if row_ids_out.dtype != torch.int32 or n_active_out.dtype != torch.int32:
        raise ValueError("row_ids_out and n_active_out must be int32")
    if row_ids_out.numel() < state.capacity or n_active_out.numel() < 1:
        raise ValueError("row_ids_out must hold capacity entries and n_active_out one")
    _check(lib().espo_compact_active(state.handle, _dev_ptr(row_ids_out, "row_ids_out"),
                                     _dev_ptr(n_active_out, "n_active_out"), _stream(stream)), "espo_compact_active")


def espo_end_batch(state: EspoState, params: espo_params, alpha_ema: float = 0.99, eta_beta: float = 0.1,
                   tau: float = 0.25, beta_min: float = 0.0, beta_max: float = 3.0e38, first_update: bool = False,
                   stream=None) -> dict:
    """Batch-boundary update (Eq. 7-8, 12): rewrites params.mu_g, params.sigma2_g and params.beta in place and
    returns the batch statistics; see ``espo.h``.  Synchronises the stream."""
    out = (C.c_double * 6)()
    _check(lib().espo_end_batch(state.handle, alpha_ema, eta_beta, tau, beta_min, beta_max, int(bool(first_update)),
                                C.byref(params), out, _stream(stream)), "espo_end_batch")
    return {"mean_g": out[0], "var_g": out[1], "stop_rate": out[2], "tokens": int(out[3]), "trajectories": int(out[4]),
            "stopped": int(round(out[5]))}


STATS_KEYS = ("mean_g", "var_g", "stop_rate", "tokens", "trajectories", "stopped")


def espo_end_batch_merge(parts, params: espo_params, alpha_ema: float = 0.99, eta_beta: float = 0.1, tau: float = 0.25,
                         beta_min: float = 0.0, beta_max: float = 3.0e38, first_update: bool = False) -> dict:
    """Batch-boundary update from the statistics of several parts of one rollout batch (one per GPU): ``parts`` is a
    sequence of the dicts ``espo_end_batch`` returns (or of 6-number rows in that order); see ``espo.h``.  Host only."""
    rows = [[float(p[k]) for k in STATS_KEYS] if isinstance(p, dict) else [float(x) for x in p] for p in parts]
    if any(len(r) != 6 for r in rows):
        raise ValueError("every part needs six numbers: mean, variance, stop rate, tokens, trajectories, stopped")
    flat = (C.c_double * (6 * len(rows)))(*[x for r in rows for x in r])
    out = (C.c_double * 6)()
    _check(lib().espo_end_batch_merge(flat, len(rows), alpha_ema, eta_beta, tau, beta_min, beta_max, int(bool(first_update)),
                                      C.byref(params), out), "espo_end_batch_merge")
    return {"mean_g": out[0], "var_g": out[1], "stop_rate": out[2], "tokens": int(out[3]), "trajectories": int(out[4]),
            "stopped": int(round(out[5]))}


def espo_state_status(state: EspoState, stream=None) -> int:
    out = C.c_uint32(0)
    _check(lib().espo_state_status(state.handle, C.byref(out), _stream(stream)), "espo_state_status")
    return out.value


def espo_advantages_returns(rewards: torch.Tensor, values: torch.Tensor, lengths: torch.Tensor, stopped: torch.Tensor,
                            gamma: float, lam: float, r_fail: float, adv_out: torch.Tensor,
                            returns_out: Optional[torch.Tensor] = None, total_tokens: Optional[int] = None,
                            stream=None) -> None:
    """TD + GAE over packed ragged trajectories with the failure transition (Eq. 4-5, 13), and optionally the
    value targets A_t + V_t in the same pass; see ``espo.h``."""
    for t, n, dt in ((rewards, "rewards", torch.float32), (values, "values", torch.float32),
                     (adv_out, "adv_out", torch.float32), (lengths, "lengths", torch.int32),
                     (stopped, "stopped", torch.uint8)) + (() if returns_out is None else
                                                          ((returns_out, "returns_out", torch.float32),)):
        if t.dtype != dt or not t.is_contiguous():
            raise ValueError(f"{n} must be a contiguous {dt} tensor")
    total = rewards.numel() if total_tokens is None else total_tokens
    if values.numel() < total or adv_out.numel() < total or rewards.numel() < total or \
            (returns_out is not None and returns_out.numel() < total):
        raise ValueError("rewards, values and the outputs must hold total_tokens entries")
    if stopped.numel() < lengths.numel():
        raise ValueError("stopped is shorter than lengths")
    _check(lib().espo_advantages_returns(_dev_ptr(rewards, "rewards"), _dev_ptr(values, "values"),
                                         _dev_ptr(lengths, "lengths"), _dev_ptr(stopped, "stopped"), lengths.numel(),
                                         total, gamma, lam, r_fail, _dev_ptr(adv_out, "adv_out"),
                                         _dev_ptr(returns_out, "returns_out"), _stream(stream)),
           "espo_advantages_returns")


def espo_advantages_padded(rewards: torch.Tensor, values: torch.Tensor, lengths: torch.Tensor, stopped: torch.Tensor,
                           gamma: float, lam: float, r_fail: float, adv_out: torch.Tensor,
                           returns_out: Optional[torch.Tensor] = None, stream=None) -> None:
    """TD + GAE (Eq. 4-5, 13) over a padded batch: ``rewards``, ``values`` and the outputs are [B, t_max]; see ``espo.h``."""
    if rewards.dim() != 2:
        raise ValueError("rewards must be [B, t_max]")
    B, t_max = rewards.shape
    for t, n in ((rewards, "rewards"), (values, "values"), (adv_out, "adv_out")) + \
            (() if returns_out is None else ((returns_out, "returns_out"),)):
        if t.dtype != torch.float32 or not t.is_contiguous() or tuple(t.shape) != (B, t_max):
            raise ValueError(f"{n} must be a contiguous float32 [B, t_max] tensor")
    if lengths.dtype != torch.int32 or not lengths.is_contiguous() or lengths.numel() != B:
        raise ValueError("lengths must be a contiguous int32 [B] tensor")
    if stopped.dtype != torch.uint8 or not stopped.is_contiguous() or stopped.numel() < B:
        raise ValueError("stopped must be a contiguous uint8 [B] tensor")
    _check(lib().espo_advantages_padded(_dev_ptr(rewards, "rewards"), _dev_ptr(values, "values"),
                                        _dev_ptr(lengths, "lengths"), _dev_ptr(stopped, "stopped"), B, t_max,
                                        gamma, lam, r_fail, _dev_ptr(adv_out, "adv_out"),
                                        _dev_ptr(returns_out, "returns_out"), _stream(stream)),
           "espo_advantages_padded")


def espo_advantages_stats(rewards: torch.Tensor, values: torch.Tensor, lengths: torch.Tensor, stopped: torch.Tensor,
                          gamma: float, lam: float, r_fail: float, adv_out: torch.Tensor, stats_out: torch.Tensor,
                          returns_out: Optional[torch.Tensor] = None, total_tokens: Optional[int] = None,
                          stream=None) -> None:
    """espo_advantages_returns that also leaves sum A_t and sum A_t^2 in ``stats_out`` (float64 [2]); see ``espo.h``."""
    for t, n, dt in ((rewards, "rewards", torch.float32), (values, "values", torch.float32),
                     (adv_out, "adv_out", torch.float32), (lengths, "lengths", torch.int32),
                     (stopped, "stopped", torch.uint8), (stats_out, "stats_out", torch.float64)) + \
            (() if returns_out is None else ((returns_out, "returns_out", torch.float32),)):
        if t.dtype != dt or not t.is_contiguous():
            raise ValueError(f"{n} must be a contiguous {dt} tensor")
    total = rewards.numel() if total_tokens is None else total_tokens
    if values.numel() < total or adv_out.numel() < total or rewards.numel() < total or \
            (returns_out is not None and returns_out.numel() < total):
        raise ValueError("rewards, values and the outputs must hold total_tokens entries")
    if stopped.numel() < lengths.numel():
        raise ValueError("stopped is shorter than lengths")
    if stats_out.numel() < 2:
        raise ValueError("stats_out must hold two float64")
    _check(lib().espo_advantages_stats(_dev_ptr(rewards, "rewards"), _dev_ptr(values, "values"),
                                       _dev_ptr(lengths, "lengths"), _dev_ptr(stopped, "stopped"), lengths.numel(),
                                       total, gamma, lam, r_fail, _dev_ptr(adv_out, "adv_out"),
                                       _dev_ptr(returns_out, "returns_out"), _dev_ptr(stats_out, "stats_out"),
                                       _stream(stream)),
           "espo_advantages_stats")


def espo_advantages(rewards: torch.Tensor, values: torch.Tensor, lengths: torch.Tensor, stopped: torch.Tensor,
                    gamma: float, lam: float, r_fail: float, adv_out: torch.Tensor,
                    total_tokens: Optional[int] = None, stream=None) -> None:
    """TD + GAE over packed ragged trajectories with the failure transition (Eq. 4-5, 13); see ``espo.h``."""
    for t, n, dt in ((rewards, "rewards", torch.float32), (values, "values", torch.float32),
                     (adv_out, "adv_out", torch.float32), (lengths, "lengths", torch.int32),
                     (stopped, "stopped", torch.uint8)):
        if t.dtype != dt or not t.is_contiguous():
            raise ValueError(f"{n} must be a contiguous {dt} tensor")
    total = rewards.numel() if total_tokens is None else total_tokens
    if values.numel() < total or adv_out.numel() < total or rewards.numel() < total:
        raise ValueError("rewards, values and adv_out must hold total_tokens entries")
    if stopped.numel() < lengths.numel():
        raise ValueError("stopped is shorter than lengths")
    _check(lib().espo_advantages(_dev_ptr(rewards, "rewards"), _dev_ptr(values, "values"),
                                 _dev_ptr(lengths, "lengths"), _dev_ptr(stopped, "stopped"), lengths.numel(), total,
                                 gamma, lam, r_fail, _dev_ptr(adv_out, "adv_out"), _stream(stream)),
           "espo_advantages")


ESPO_NOALLOC_MAX_B, ESPO_NOALLOC_MAX_TOKENS = 4096, 1 << 24


def espo_advantages_noalloc(rewards: torch.Tensor, values: torch.Tensor, lengths: torch.Tensor, stopped: torch.Tensor,
                            gamma: float, lam: float, r_fail: float, adv_out: torch.Tensor,
                            status_out: Optional[torch.Tensor] = None, total_tokens: Optional[int] = None,
                            stream=None) -> None:
    """``espo_advantages`` for processes that cannot allocate device memory (the engine owns it all, or a
    cudaMalloc's device-wide synchronisation is not acceptable): the library's scratch is a fixed array inside
    the library image.  At most ESPO_NOALLOC_MAX_B trajectories and ESPO_NOALLOC_MAX_TOKENS tokens per call.
    ``status_out`` (int32/uint32 CUDA tensor of one element, or None) receives the ESPO_DEV_* bits."""
    for t, n, dt in ((rewards, "rewards", torch.float32), (values, "values", torch.float32),
                     (adv_out, "adv_out", torch.float32), (lengths, "lengths", torch.int32),
                     (stopped, "stopped", torch.uint8)):
        if t.dtype != dt or not t.is_contiguous():
            raise ValueError(f"{n} must be a contiguous {dt} tensor")
    total = rewards.numel() if total_tokens is None else total_tokens
    if values.numel() < total or adv_out.numel() < total or rewards.numel() < total:
        raise ValueError("rewards, values and adv_out must hold total_tokens entries")
    if stopped.numel() < lengths.numel():
        raise ValueError("stopped is shorter than lengths")
    if status_out is not None and (status_out.element_size() != 4 or status_out.numel() < 1):
        raise ValueError("status_out must hold one 32-bit word")
    _check(lib().espo_advantages_noalloc(_dev_ptr(rewards, "rewards"), _dev_ptr(values, "values"),
                                         _dev_ptr(lengths, "lengths"), _dev_ptr(stopped, "stopped"),
                                         lengths.numel(), total, gamma, lam, r_fail, _dev_ptr(adv_out, "adv_out"),
                                         _dev_ptr(status_out, "status_out"), _stream(stream)),
           "espo_advantages_noalloc")


def espo_advantages_reserve(max_B: int, max_tokens: int) -> None:
    _check(lib().espo_advantages_reserve(max_B, max_tokens), "espo_advantages_reserve")


def espo_advantages_status(stream=None) -> int:
    out = C.c_uint32(0)
    _check(lib().espo_advantages_status(C.byref(out), _stream(stream)), "espo_advantages_status")
    return out.value
