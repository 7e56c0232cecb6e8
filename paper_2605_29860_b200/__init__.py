"""B200-native (sm_100a) implementation of ESPO's per-decode-step early-stopping hot path
and its truncated-trajectory GAE pass, behind the C ABI declared in ``include/espo.h``.

``binding`` exposes the C entry points under the same names; ``synth`` holds the seeded
synthetic-input generators used by the tests and the benchmark (no method arithmetic).
"""
from .binding import (  # noqa: F401
    ESPO_ERR_ALIGN, ESPO_ERR_BAD_DTYPE, ESPO_ERR_BAD_PARAM, ESPO_ERR_BAD_SHAPE, ESPO_ERR_CAPACITY, ESPO_ERR_CUDA,
    ESPO_ERR_NULL, ESPO_OK,
    ESPO_BF16, ESPO_DEV_BAD_LENGTHS, ESPO_DEV_BAD_ROW, ESPO_DEV_BAD_SLOT, ESPO_DEV_NAN_VALUE, ESPO_DEV_TIMEOUT,
    ESPO_F32, ESPO_NOALLOC_MAX_B, ESPO_NOALLOC_MAX_TOKENS, ESPO_ROW_ACTIVE, ESPO_ROW_BAD, ESPO_ROW_EOS, ESPO_ROW_STOPPED, ESPO_ROW_TMAX, ESPO_SAMPLER_FLAT,
    ESPO_SAMPLER_HIER, ESPO_STOP_ESPO, ESPO_STOP_RANDOM, ESPO_STOP_REGRET_ONLY, ESPO_STOP_VALUE_ONLY, EspoError, EspoState, espo_advantages, espo_advantages_noalloc, espo_advantages_padded, espo_advantages_reserve, espo_advantages_returns, espo_advantages_stats, espo_advantages_status,
    espo_compact_active, espo_end_batch, espo_end_batch_merge, espo_free_state, espo_init_state, espo_params, espo_reset_state, espo_set_dependent_launch, espo_set_launch_config,
    espo_state_status, espo_state_view, espo_step, espo_step_merge, espo_step_partial, make_params)
