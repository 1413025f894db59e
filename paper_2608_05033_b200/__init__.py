"""Structure-adaptive SpMM for B200 (sm_100a): thin Python binding over libsd.so.

Importing the package does not load the shared library; the first call does,
and it raises if the library has not been built.
"""
from .binding import (  # noqa: F401
    SD_OK, SD_ERR_INVALID_ARG, SD_ERR_UNSUPPORTED, SD_ERR_ALLOC, SD_ERR_CUDA, SD_ERR_INTERNAL,
    SD_F32, SD_BF16, SD_AUTO, SD_ROWSPLIT, SD_MERGE, SD_BSR_TC, SD_HYBRID, FAMILY_NAMES, EXPORTS,
    Plan, SdError, load, sd_plan_create, sd_plan_create_ex, sd_spmm, sd_spmm_host, sd_spmm_host_async, sd_plan_sync, sd_plan_update_values, sd_plan_save, sd_plan_load, sd_plan_destroy,
    sd_plan_get_info, sd_plan_get_features, sd_features_t, SHAPE_NAMES, sd_plan_get_bsr, sd_plan_get_tiles, sd_plan_get_segments, sd_plan_get_hybrid, sd_plan_device_status, sd_spmm_merge_static, sd_last_error, sd_plan_desc_t, sd_plan_info_t,
)
