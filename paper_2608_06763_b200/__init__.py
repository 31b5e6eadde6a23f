"""B200 (sm_100a) CubicQuant packed-weight GEMV/GEMM: thin Python binding of libcubicquant.so.

Every function here only marshals arguments (torch tensors -> device pointers, current CUDA
stream) into the C ABI declared in include/cubicquant.h; all arithmetic runs in the CUDA
kernels.  There is no CPU fallback: importing works without a GPU (so the build can be checked),
but every compute call needs a CUDA device and the built shared library.
"""
from .binding import (CQ_DYN_A8, CQ_EFFORT, CQ_FIT_CONTINUOUS, CQ_FIT_JOINT, CQ_MODEL_DTYPE, CubicQuantError, PackedWeights, cq_canonical_code_bytes,
                      cq_debug_a8_partials, cq_debug_gemm_plan, cq_debug_wait_timeout, cq_decode_carriers, cq_decode_levels, cq_decode_weights,
                      cq_effective_bits, cq_encode, cq_encode_assign, cq_encode_losses, cq_encode_scale, cq_gemm, cq_gemm_host, cq_gemm_routed, cq_gemm_status, cq_gemv_static, cq_layout_bytes, cq_mlp_swiglu, cq_pack_codes, cq_quantize_a8,
                      cq_repack, cq_status_string, cq_unpack, cq_workspace_bytes, cq_workspace_init, lib,
                      library_path)

__all__ = [n for n in dir() if n.startswith(("cq_", "CQ_"))] + ["PackedWeights", "CubicQuantError", "lib",
                                                                  "library_path"]
