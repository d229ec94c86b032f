"""B200-native R-KV decode-time KV-cache compression step (C-ABI CUDA library + thin ctypes binding).

Every step of the path runs in the CUDA kernels of ``librkv_b200.so``; this package only marshals
arguments.  There is no CPU fallback: loading fails loudly if the library has not been built.
"""
from .binding import (  # noqa: F401
    RKV_BF16, RKV_F32, RKV_FP8_E4M3, RKV_FLAG_SIMT_SCORES, RKV_FLAG_ROWBLOCK_SCORES, RKV_FLAG_MEAN_THEN_POOL, RKV_FLAG_HEAD_MEAN, RKV_FLAG_GQA_MEAN_POOL, RKV_FLAG_NO_SYMMETRIC, RKV_STAGE_ALL, RKV_STAGE_GATHER, RKV_STAGE_PREP,
    RKV_STAGE_SCORES, RKV_STAGE_SELECT, RKV_OK, RkvDesc, RkvError, Compressor, lib, lib_path,
    rkv_compress, rkv_compress_ex, rkv_compress_stages, rkv_compress_host, rkv_compress_static,
    RKV_STATIC_SCRATCH_BYTES, rkv_desc_default, rkv_append, rkv_push_query, rkv_selftest_wait_expiry, rkv_decode_attention, rkv_decode_workspace_bytes,
    rkv_host_workspace_bytes, rkv_launch_count, rkv_launch_count_for, rkv_set_desc, rkv_status_string, rkv_workspace_bytes,
)
