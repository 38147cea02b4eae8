"""B200-native streamFFN routed-expert path (CascadeEP prefill MoE layer).

The product is the C-ABI library ``libcascade_ffn.so`` (CUDA, sm_100a); this package
is its thin Python binding (argument marshalling only) plus the seeded input
generator used by the tests and the benchmark.
"""
from . import workloads  # noqa: F401
from .binding import (CepConfig, CepError, InvocationInfo, MoELayer, lib, load_library,  # noqa: F401
                      moe_plan_workspace_bytes, moe_packed_weight_bytes, moe_plan, moe_load_weights,
                      ffn_begin, ffn_set_addend, moe_route, ffn_submit_chunk, ffn_flush, combine, ffn_status, ffn_num_invocations, ffn_wait_invocation,
                      ffn_query, ffn_query_call, ffn_debug_export, cep_kernel_launches, moe_plan_destroy, cep_last_error,
                      cep_debug_decode_tile, cep_debug_schedule, layout_indices_noalloc, cep_debug_wait_timeout, cep_debug_check_guards,
                      ffn_set_active_streams, cep_calibrate, cep_calibrate_routed,
                      CEP_BF16, CEP_FP8_E4M3_BLOCK128, CEP_MXFP4_E4M3, DTYPE_OF, CEP_MODE_SYNC, CEP_MODE_ASYNC, CEP_MODE_STREAMFFN,
                      CEP_GEMM_TCGEN05, CEP_GEMM_SIMT, CEP_GEMM_TCGEN05_1CTA, STATUS_NAMES)
