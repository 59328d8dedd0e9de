"""B200 (sm_100a) HLQ look-up-table GEMM/GEMV: thin Python binding over the C-ABI library.

Every step of the path runs in the CUDA kernels of `libelutq.so`; this package only
marshals torch tensors (device memory, streams) into the C calls declared in
`include/elutq.h`.  There is no CPU fallback: a missing library raises.
"""

from .binding import (  # noqa: F401
    ElutqError,
    FLAG_SKIP_OFFSET,
    FLAG_OFFSET_ONLY,
    FLAG_OUT_F32,
    FLAG_ACCUMULATE,
    FLAG_PLAIN_G4,
    FLAG_CLUSTER_REDUCE,
    FLAG_MIRROR,
    FLAG_LUT_ONLY,
    FLAG_TABLE_F16,
    FLAG_TABLE_I8,
    GemvCall,
    lib,
    library_path,
    elutq_packed_bytes,
    elutq_pack,
    elutq_unpack,
    elutq_describe,
    elutq_forget,
    elutq_workspace_bytes,
    elutq_workspace_init,
    elutq_lut_gemm,
    elutq_lut_gemm_bias,
    elutq_lut_gemm_f32,
    elutq_lut_gemm_ws,
    elutq_lut_gemm_host,
    elutq_lut_gemm_static,
    elutq_hlq_fit,
    elutq_chain_plan_bytes,
    elutq_chain_plan,
    elutq_chain_run,
    elutq_chain_run_opts,
    elutq_chain_status,
    elutq_chain_forget,
    elutq_device_status,
    elutq_launch_count,
    elutq_release_scratch,
    elutq_status_string,
    elutq_last_cuda_error,
)
