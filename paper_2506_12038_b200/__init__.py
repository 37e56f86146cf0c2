"""B200-native LUT-based inference matmul (LCD paper, Section 4) behind a C ABI.

`binding` loads liblcd_b200.so (built in-tree by `build.py`) and fails loudly if it is absent.
"""
from .binding import (ActBatch, FusedBatch, HostBatch, LinearBatch, MAX_BATCH, ALGO_AUTO, ALGO_BUCKET_LUT, ALGO_DENSE_F16, ALGO_DENSE_TC, ALGO_REFERENCE, ALGO_REGISTER_LUT, ALGO_TC_LUT, ALGO_SHARED_BUCKET, LcdError,  # noqa: F401
                      PackedWeights, linear_host, linear_host_scratch_bytes, lut_linear, lut_linear_static,
                      lut_linear_workspace_bytes, resolve_batch_algo, pack_weights, packed_weights_bytes, smooth_quantize_act, smoothing_search, reclassify, dbci,
                      unpack_weights)
