"""Transposable N:M mask search on NVIDIA B200: Python binding of the C-ABI CUDA library.

The binding only marshals arguments (torch tensors -> device pointers); every step of the search
runs in the CUDA kernels of ``libtm.so``.  There is no CPU fallback: a missing library or a missing
CUDA device raises.
"""
from .binding import (  # noqa: F401
    TM_APPROX, TM_APPROX_COVER, TM_BF16, TM_DEV_INTERNAL, TM_DEV_NONFINITE, TM_EXACT, TM_F32,
    TmBatch, TmError, TmPlan, tm_plan_create, tm_plan_run, tm_plan_destroy, library_path, load_library, tm_device_status, tm_find_mask, tm_find_mask_batched, tm_find_mask_batched_static, TM_STATIC_MAX_MATRICES,
    tm_find_mask_bf16, tm_find_mask_host, tm_mask_words, tm_mask_words_per_row, tm_status_string,
    tm_version, tm_workspace_bytes, tm_aux_workspace_bytes, tm_nm_mask_1d, tm_mask_violations, tm_mask_hamming, tm_compress_2_4,
    TM_DEV_BADMASK, TM_NM1D_ABSORB_MEAN,
)
