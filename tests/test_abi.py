"""The C-ABI library loads and exports every entry point that include/espo.h declares (CPU only)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    src = open(os.path.join(ROOT, "include", "espo.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(espo_[a-z_0-9]+)\s*\(", src)))


@pytest.fixture(scope="module")
def lib():
    from paper_2605_29860_b200 import build
    return ctypes.CDLL(build.build())


def test_header_declares_the_documented_entry_points():
    names = _declared_functions()
    for must in ("espo_init_state", "espo_step", "espo_advantages", "espo_reset_state", "espo_free_state",
                 "espo_state_view", "espo_compact_active", "espo_state_status", "espo_strerror"):
        assert must in names


def test_every_declared_symbol_is_exported(lib):
    for name in _declared_functions():
        assert hasattr(lib, name), f"{name} is declared in espo.h but not exported by libespo.so"


def test_argument_errors_are_reported_without_a_device(lib):
    # these paths return before any CUDA call is made
    lib.espo_strerror.restype = ctypes.c_char_p
    assert lib.espo_strerror(0) == b"ok"
    for code in range(-7, 0):
        assert lib.espo_strerror(code) and b"unknown error code" not in lib.espo_strerror(code)
    assert b"unknown error code" in lib.espo_strerror(-99)
    lib.espo_init_state.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_uint64,
                                    ctypes.c_uint64, ctypes.c_void_p]
    assert lib.espo_init_state(None, 1, 1, 0, 0, None) == -1                    # NULL out pointer
    h = ctypes.c_void_p()
    assert lib.espo_init_state(ctypes.byref(h), 0, 10, 0, 0, None) == -3         # capacity < 1
    assert lib.espo_init_state(ctypes.byref(h), 4, 0, 0, 0, None) == -3          # V < 1
    assert lib.espo_init_state(ctypes.byref(h), 4, 10, 0, 1 << 30, None) == -7   # batch_id too large
    assert lib.espo_step(None, 0, 0, None, 0, None, 0, None, None, None, None, None) == -1
    assert lib.espo_reset_state(None, 0, None) == -1
    assert lib.espo_state_status(None, None, None) == -1
    assert lib.espo_compact_active(None, None, None, None) == -1
    assert lib.espo_advantages_status(None, None) == -1
    lib.espo_free_state(None)                                                    # ignored


def test_python_binding_mirrors_the_abi():
    import paper_2605_29860_b200 as espo
    for name in _declared_functions():
        if name == "espo_strerror" or name == "espo_last_cuda_error":
            continue
        assert hasattr(espo, name), f"binding lacks {name}"
    assert ctypes.sizeof(espo.espo_params) == 76


def test_end_batch_merge_pools_the_parts_statistics(lib):
    # host-only entry point: pooled mean / population variance / stop rate of parts given by (mean, var, rho, n, traj, stopped)
    import numpy as np
    import paper_2605_29860_b200 as espo
    rng = np.random.default_rng(0)
    groups = [rng.gamma(2.0, 1.5, size=n) for n in (1200, 1, 35000)]
    traj, stopped = [40, 1, 300], [10, 0, 77]
    parts = [[g.mean(), g.var(), s / t, g.size, t, s] for g, t, s in zip(groups, traj, stopped)] + [[0.0, 0.0, 0.0, 0, 0, 0]]
    allg = np.concatenate(groups)
    for first in (False, True):
        p = espo.make_params(mu_g=2.0, sigma2_g=3.0, beta=7.0)
        st = espo.espo_end_batch_merge(parts, p, alpha_ema=0.9, eta_beta=0.5, tau=0.25, beta_min=0.0, beta_max=7.05,
                                       first_update=first)
        rho = sum(stopped) / sum(traj)
        assert abs(st["mean_g"] - allg.mean()) < 1e-12 and abs(st["var_g"] - allg.var()) < 1e-10 and abs(st["stop_rate"] - rho) < 1e-15
        assert (st["tokens"], st["trajectories"], st["stopped"]) == (allg.size, sum(traj), sum(stopped))
        want_mu = allg.mean() if first else 0.9 * 2.0 + 0.1 * allg.mean()              # Eq. 7
        want_s2 = allg.var() if first else 0.9 * 3.0 + 0.1 * allg.var()                # Eq. 8
        want_beta = min(max(7.0 + 0.5 * (rho - 0.25), 0.0), 7.05)                      # Eq. 12, clipped
        assert abs(p.mu_g - want_mu) < 1e-6 and abs(p.sigma2_g - want_s2) < 1e-6 and abs(p.beta - want_beta) < 1e-6
    q = espo.make_params(mu_g=2.0, sigma2_g=3.0, beta=7.0)
    espo.espo_end_batch_merge([[0.0] * 6], q)                                          # no tokens: nothing changes
    assert (q.mu_g, q.sigma2_g, q.beta) == (2.0, 3.0, 7.0)
    import pytest
    with pytest.raises(espo.EspoError):
        espo.espo_end_batch_merge([[1.0, 1.0, 0.0, -5, 1, 0]], q)
