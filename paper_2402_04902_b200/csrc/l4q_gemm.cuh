#pragma once
#include "l4q_common.cuh"
namespace l4q {
inline l4q_status gemm_forward_bf16(const Params&, const void*, const void*, void*, cudaStream_t, int* n) { *n = 0; return L4Q_ERR_UNSUPPORTED; }
inline l4q_status gemm_dgrad_bf16(const Params&, const void*, const void*, void*, cudaStream_t, int* n) { *n = 0; return L4Q_ERR_UNSUPPORTED; }
inline l4q_status gemm_wgrad_bf16(const Params&, const void*, const void*, const void*, const float*, const float*, const float*, const float*, float*, float*, float*, float*, cudaStream_t, int* n) { *n = 0; return L4Q_ERR_UNSUPPORTED; }
}
