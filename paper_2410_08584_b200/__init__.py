"""ZipVL per-layer hot path for NVIDIA B200 (sm_100a): Python binding.

``libzipvl.so`` (hand-written CUDA behind a C ABI, see ``include/zipvl.h``) does
all the work; this package marshals torch tensors into it.  Importing the
package does not load the library; the first call (or ``load()``) does, and
raises if it has not been built -- there is no CPU or PyTorch fallback.
"""
from . import workloads
from .binding import (BUDGET_BY_NORM, DEV_BAD_INDEX, DEV_BAD_VALUE, DEV_CAPACITY, DEV_TIMEOUT, EXPORTS, LIB_PATH,
                      OP_COMPACT_KV, OP_DECODE, OP_SCORE, OP_SELECT, OP_SPARSE_PREFILL,
                      OUT_COMPACT, OUT_PADDED, TOPK_BY_ACC, ZIPVL_BF16, ZIPVL_F16, ZIPVL_F32, ZipvlError,
                      keep_last, layer_desc, load, workspace, zipvl_compact_kv, zipvl_decode, zipvl_sparse_prefill_compact,
                      QuantCache, zipvl_decode_desc, zipvl_decode_noalloc, zipvl_decode_paged, zipvl_decode_quant, zipvl_decode_quant_batch, quant_cache_table, zipvl_quantize_kv, zipvl_launch_count, zipvl_layer, zipvl_layer_step_host, zipvl_prefill_layer_host, zipvl_release_host_scratch, zipvl_score,
                      zipvl_batch, zipvl_score_batch, zipvl_select, zipvl_select_batch, zipvl_sparse_prefill_batch, zipvl_selftest_wait_timeout, zipvl_sparse_prefill, zipvl_workspace_bytes)

__all__ = [n for n in dir() if not n.startswith("_")]
