"""ctypes loader for the ESPO reference oracle (``espo_oracle.cpp``).

TEST INFRASTRUCTURE ONLY.  The oracle is a slow double-precision CPU statement of
the method, written from the paper's equations (Sec. 3 Eq. 4-5, Sec. 4 Eq. 6-13,
Algorithm 1).  Nothing in the product package imports this module; only the tests,
the smoke check and the benchmark's CPU-baseline leg do.  It shares no code with
the CUDA library.

The shared object is compiled on first use with ``g++`` (plain C++17, no CUDA).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "espo_oracle.cpp")
_SO = os.path.join(_HERE, "libespo_oracle.so")
_lock = threading.Lock()
_lib = None

ACTIVE, STOPPED, EOS, TMAX, BAD = 0, 1, 2, 3, 4
SAMPLER_FLAT, SAMPLER_HIER = 0, 1
STOP_ESPO, STOP_VALUE_ONLY, STOP_REGRET_ONLY, STOP_RANDOM = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile ``espo_oracle.cpp`` into ``libespo_oracle.so`` next to it (if stale)."""
    with _lock:
        stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _SO + f".tmp{os.getpid()}"
            cmd = ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-pthread",
                   "-ffp-contract=off", "-o", tmp, _SRC]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _SO)
    return _SO


class Params(C.Structure):
    """Frozen per-batch parameters (Eq. 9-11, Algorithm 1 inputs)."""
    _fields_ = [("temperature", C.c_double), ("mu_g", C.c_double), ("sigma2_g", C.c_double),
                ("delta", C.c_double), ("clip_c", C.c_double), ("alpha_s", C.c_double),
                ("beta", C.c_double), ("eps", C.c_double), ("warmup_complete", C.c_int32),
                ("t_max", C.c_int32), ("eos_token", C.c_int32), ("sampler", C.c_int32),
                ("stop_mode", C.c_int32), ("shadow", C.c_int32), ("tau", C.c_double), ("p_random", C.c_double),
                ("top_p", C.c_double), ("top_k", C.c_int32), ("pad_", C.c_int32)]


class RowState(C.Structure):
    _fields_ = [("z", C.c_double), ("sum_g", C.c_double), ("sum_g2", C.c_double),
                ("n_tokens", C.c_int64), ("t", C.c_int32), ("status", C.c_int32),
                ("t_stop", C.c_int32), ("pad_", C.c_int32)]


class StepOut(C.Structure):
    _fields_ = [("g", C.c_double), ("g_tilde", C.c_double), ("z", C.c_double), ("logp", C.c_double),
                ("max_x", C.c_double), ("log_s", C.c_double), ("min_rel_gap", C.c_double),
                ("threshold", C.c_double), ("entropy", C.c_double), ("token", C.c_int32), ("stop", C.c_int32),
                ("runner_up", C.c_int32), ("bad", C.c_int32), ("filter_margin", C.c_double), ("kept", C.c_int64)]


def make_params(temperature=1.0, mu_g=0.0, sigma2_g=1.0, delta=1e-8, clip_c=10.0, alpha_s=0.9,
                beta=7.0, eps=0.2, warmup_complete=1, t_max=8192, eos_token=-1, sampler=SAMPLER_FLAT,
                stop_mode=0, shadow=0, tau=0.0, p_random=0.0, top_p=1.0, top_k=0) -> Params:
    return Params(float(temperature), float(mu_g), float(sigma2_g), float(delta), float(clip_c),
                  float(alpha_s), float(beta), float(eps), int(warmup_complete), int(t_max),
                  int(eos_token), int(sampler), int(stop_mode), int(shadow), float(tau), float(p_random),
                  float(top_p), int(top_k), 0)


def lib():
    global _lib
    if _lib is None:
        so = build()
        L = C.CDLL(so)
        dp, ip, u8p, u32p, fp = (C.POINTER(C.c_double), C.POINTER(C.c_int32), C.POINTER(C.c_uint8),
                                 C.POINTER(C.c_uint32), C.POINTER(C.c_float))
        L.espo_oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.espo_oracle_philox4x32_10.restype = None
        L.espo_oracle_uniform.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint32, C.c_int, C.c_uint64]
        L.espo_oracle_uniform.restype = C.c_double
        L.espo_oracle_init_row.argtypes = [C.POINTER(RowState)]
        L.espo_oracle_init_row.restype = None
        L.espo_oracle_log_softmax.argtypes = [dp, C.c_int64, C.c_double, dp]
        L.espo_oracle_log_softmax.restype = None
        L.espo_oracle_step_row.argtypes = [dp, C.c_int64, C.c_double, C.c_uint64, C.c_uint64, C.c_uint32,
                                           C.POINTER(Params), C.c_int32, C.POINTER(RowState), C.POINTER(StepOut)]
        L.espo_oracle_step_row.restype = None
        L.espo_oracle_step_batch.argtypes = [dp, C.c_int64, dp, ip, C.c_int32, C.c_uint64, C.c_uint64,
                                             C.POINTER(Params), ip, C.POINTER(RowState), C.POINTER(StepOut),
                                             C.c_int32]
        L.espo_oracle_step_batch.restype = None
        L.espo_oracle_step_batch_f32.argtypes = [fp, C.c_int64, dp, ip, C.c_int32, C.c_uint64, C.c_uint64,
                                                 C.POINTER(Params), C.POINTER(RowState), C.POINTER(StepOut),
                                                 C.c_int32]
        L.espo_oracle_step_batch_f32.restype = None
        for name in ("espo_oracle_advantages", "espo_oracle_advantages_direct"):
            fn = getattr(L, name)
            fn.argtypes = [dp, dp, ip, u8p, C.c_int32, C.c_double, C.c_double, C.c_double, dp]
            fn.restype = None
        L.espo_oracle_end_batch.argtypes = [C.POINTER(RowState), C.c_int32, C.c_double, C.c_double, C.c_double,
                                            C.c_double, C.c_double, C.c_int32, dp, dp, dp, dp]
        L.espo_oracle_end_batch.restype = None
        L.espo_oracle_advantages_f32.argtypes = [fp, fp, ip, u8p, C.c_int32, C.c_double, C.c_double,
                                                 C.c_double, dp, C.c_int32]
        L.espo_oracle_advantages_f32.restype = None
        _lib = L
    return _lib


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().espo_oracle_philox4x32_10(_ptr(c, C.c_uint32), _ptr(k, C.c_uint32), _ptr(out, C.c_uint32))
    return out


def uniform(seed, batch_id, slot, step, level, index) -> float:
    return float(lib().espo_oracle_uniform(int(seed), int(batch_id), int(slot), int(step), int(level), int(index)))


def log_softmax(logits, temperature=1.0) -> np.ndarray:
    x = np.ascontiguousarray(logits, dtype=np.float64)
    out = np.empty_like(x)
    lib().espo_oracle_log_softmax(_ptr(x, C.c_double), x.size, float(temperature), _ptr(out, C.c_double))
    return out


class Rollout:
    """Per-trajectory oracle state for one rollout batch (Algorithm 1's z, t, done)."""

    def __init__(self, capacity: int, seed: int, batch_id: int = 0):
        self.capacity = int(capacity)
        self.seed = int(seed)
        self.batch_id = int(batch_id)
        self.states = (RowState * self.capacity)()
        for i in range(self.capacity):
            lib().espo_oracle_init_row(C.byref(self.states[i]))

    def step(self, logits, values, params: Params, row_ids=None, forced_tokens=None, n_threads=1):
        """Advance the listed rows by one decode step.

        ``logits`` [n_rows, V] (any float dtype; widened exactly to float64),
        ``values`` [n_rows].  Returns a list-like ctypes array of ``StepOut``.
        """
        x = np.ascontiguousarray(logits, dtype=np.float64)
        n_rows, V = x.shape
        v = np.ascontiguousarray(values, dtype=np.float64)
        rid = None if row_ids is None else np.ascontiguousarray(row_ids, dtype=np.int32)
        ft = None if forced_tokens is None else np.ascontiguousarray(forced_tokens, dtype=np.int32)
        outs = (StepOut * n_rows)()
        lib().espo_oracle_step_batch(
            _ptr(x, C.c_double), V, _ptr(v, C.c_double),
            None if rid is None else _ptr(rid, C.c_int32), n_rows, self.seed, self.batch_id,
            C.byref(params), None if ft is None else _ptr(ft, C.c_int32), self.states, outs, int(n_threads))
        return outs

    def step_f32(self, logits_f32, values, params: Params, row_ids=None, n_threads=1):
        """Same step on float32 rows without a float64 copy (timed CPU baseline)."""
        x = np.ascontiguousarray(logits_f32, dtype=np.float32)
        n_rows, V = x.shape
        v = np.ascontiguousarray(values, dtype=np.float64)
        rid = None if row_ids is None else np.ascontiguousarray(row_ids, dtype=np.int32)
        outs = (StepOut * n_rows)()
        lib().espo_oracle_step_batch_f32(
            _ptr(x, C.c_float), V, _ptr(v, C.c_double),
            None if rid is None else _ptr(rid, C.c_int32), n_rows, self.seed, self.batch_id,
            C.byref(params), self.states, outs, int(n_threads))
        return outs

    def end_batch(self, mu_g, sigma2_g, beta, alpha_ema=0.99, eta_beta=0.1, tau=0.25, beta_min=0.0, beta_max=1e30,
                  first_update=False):
        """Batch-boundary update (Eq. 7-8, 12).  Returns (mu_g, sigma2_g, beta, stats[6])."""
        m, v, b = C.c_double(mu_g), C.c_double(sigma2_g), C.c_double(beta)
        out = (C.c_double * 6)()
        lib().espo_oracle_end_batch(self.states, self.capacity, float(alpha_ema), float(eta_beta), float(tau),
                                    float(beta_min), float(beta_max), int(bool(first_update)),
                                    C.byref(m), C.byref(v), C.byref(b), out)
        return m.value, v.value, b.value, list(out)

    def snapshot(self, slot: int) -> RowState:
        s = RowState()
        C.memmove(C.byref(s), C.byref(self.states[slot]), C.sizeof(RowState))
        return s

    def restore(self, slot: int, s: RowState) -> None:
        C.memmove(C.byref(self.states[slot]), C.byref(s), C.sizeof(RowState))


def advantages(rewards, values, lengths, stopped, gamma, lam, r_fail, direct=False) -> np.ndarray:
    """GAE over packed ragged trajectories with the absorbing failure transition (Eq. 4-5, 13)."""
    r = np.ascontiguousarray(rewards, dtype=np.float64)
    v = np.ascontiguousarray(values, dtype=np.float64)
    L = np.ascontiguousarray(lengths, dtype=np.int32)
    s = np.ascontiguousarray(stopped, dtype=np.uint8)
    assert r.size == v.size == int(L.sum())
    out = np.zeros(r.size, dtype=np.float64)
    fn = lib().espo_oracle_advantages_direct if direct else lib().espo_oracle_advantages
    fn(_ptr(r, C.c_double), _ptr(v, C.c_double), _ptr(L, C.c_int32), _ptr(s, C.c_uint8), L.size,
       float(gamma), float(lam), float(r_fail), _ptr(out, C.c_double))
    return out


def advantages_padded(rewards, values, lengths, stopped, gamma, lam, r_fail, direct=False) -> np.ndarray:
    """The same pass on a padded batch: ``rewards`` and ``values`` are [B, t_max], trajectory i owns the first
    ``lengths[i]`` entries of row i (Eq. 4-5, 13 row by row).  Padding is never read (NaN there is fine) and comes
    back as 0."""
    r = np.asarray(rewards, dtype=np.float64)
    v = np.asarray(values, dtype=np.float64)
    L = np.asarray(lengths, dtype=np.int32)
    B, t_max = r.shape
    assert v.shape == r.shape and L.size == B and np.all((L >= 0) & (L <= t_max))
    valid = np.arange(t_max)[None, :] < L[:, None]
    out = np.zeros((B, t_max), dtype=np.float64)
    out[valid] = advantages(r[valid], v[valid], L, stopped, gamma, lam, r_fail, direct=direct)   # row-major: row after row
    return out


def advantages_f32(rewards, values, lengths, stopped, gamma, lam, r_fail, n_threads=1) -> np.ndarray:
    r = np.ascontiguousarray(rewards, dtype=np.float32)
    v = np.ascontiguousarray(values, dtype=np.float32)
    L = np.ascontiguousarray(lengths, dtype=np.int32)
    s = np.ascontiguousarray(stopped, dtype=np.uint8)
    out = np.zeros(r.size, dtype=np.float64)
    lib().espo_oracle_advantages_f32(_ptr(r, C.c_float), _ptr(v, C.c_float), _ptr(L, C.c_int32),
                                     _ptr(s, C.c_uint8), L.size, float(gamma), float(lam), float(r_fail),
                                     _ptr(out, C.c_double), int(n_threads))
    return out
