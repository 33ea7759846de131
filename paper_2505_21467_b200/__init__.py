"""B200-native FreeCache denoising-step kernels for diffusion language models.

The product is the C-ABI library ``libdlm.so`` (sources in ``csrc/``, interface in
``include/dlm.h``).  This package is its thin Python binding: same names, same argument order,
marshalling only.  Build the library with ``python -m paper_2505_21467_b200.build``.
"""
from ._binding import (  # noqa: F401
    DLM_OK, DLM_ERR_NULL, DLM_ERR_SHAPE, DLM_ERR_UNSUPPORTED, DLM_ERR_CAPACITY, DLM_ERR_WORKSPACE,
    DLM_ERR_CUDA, DLM_ERR_TIMEOUT, DLM_ERR_INDEX, DLM_ERR_DEVICE, DLM_DST_APPEND, DLM_DST_WINDOW, DlmError, dlm_kv_cache, lib, make_kv_cache,
    dlm_create, dlm_destroy, dlm_get_status, dlm_strerror, dlm_launch_count, dlm_selftest_wait_timeout, dlm_selftest_set_wait_limit, dlm_selftest_set_attn_team_max, dlm_selftest_attn_schedule,
    dlm_kv_cache_commit, dlm_attn_workspace_bytes, dlm_freecache_attn_step,
    dlm_unmask_workspace_bytes, dlm_unmask_select, dlm_unmask_select_static, dlm_guided_accept, dlm_guided_accept_topk,
    dlm_unmask_scored_workspace_bytes, dlm_unmask_select_scored, dlm_guided_accept_threshold,
    dlm_window_proj_workspace_bytes, dlm_window_qkv_project, dlm_window_qkv_project_rope, dlm_window_qkv_project_stage, dlm_window_out_project,
    DLM_SCORE_CONFIDENCE, DLM_SCORE_NEG_ENTROPY, DLM_SCORE_MARGIN, DLM_SCORE_LOG_CONF_PLUS_NOISE,
)
