"""ZipLine barrier-selection search (ElasticBSP, arXiv 2001.01347) as sm_100a CUDA kernels.

``binding`` loads ``libzipline.so`` (built in-tree by ``build``) and exposes the C ABI declared
in ``include/zipline.h`` under the same names.
"""
from .binding import (ZL_FLAG_CHECK_SORTED, ZL_FLAG_FULL_SWEEP, ZL_FLAG_PREDICTOR, ZL_FLAG_DEBUG_CHECKS, ZL_FLAG_FORCE_FILTER, zl_gridscan_batched, zl_predict_batched, zl_probe_read_batched, ZL_OBJ_RANGE, ZL_OBJ_SUM, ZL_OK,  # noqa: F401
                      Selection, ZipLine, ZipLineError, zl_max_workers, zl_status_string,
                      zl_noalloc_max_batch, zl_noalloc_scratch_bytes, zl_select_batched_noalloc,
                      zl_trace_batched, zl_trace_max_elements)
