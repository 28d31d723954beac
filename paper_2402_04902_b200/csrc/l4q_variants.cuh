// The two layers the paper sets L4Q against, on the same tensor-core GEMM template, so that the
// per-step cost of L4Q's merged quantization can be measured against them on the same hardware
// (Sec. 3.1; the training-time remark of App. E):
//
//   LoRA      Y = X W0^T + gamma (X A^T) B^T                                     (Eq. 1)
//             dA = gamma (dY B)^T X,  dB = gamma dY^T (X A^T)                    (Eq. 2)
//             dX = dY W0 + gamma (dY B) A
//   QAT-LoRA  the same with W0 replaced by its fake-quantized twin Q(W0) (Eq. 3), plus the LSQ
//             gradients ds, db (Eq. 5-6) of that quantizer from the full weight gradient dY^T X.
//
// The rank-side tensors are kept in bf16, padded to 64 columns (one K block of the GEMM):
//   Xt  = X A^T  [tokens, 64]      dYt = dY B  [tokens, 64]
//   Ab  = A      [64, d_in]        gAb = gamma A      (rows >= rank are zero)
//   Bb  = B      [d_out, 64]       gBb = gamma B      (columns >= rank are zero)
// and the LoRA path joins the main product inside the accumulator as one more K block:
//   Y  = [X | Xt]  [W | gBb]^T          dX = [dY | dYt] [W ; gAb]
#pragma once

#include "l4q_gemm.cuh"

namespace l4q {

constexpr int LORA_PAD = 64;      // padded rank = one K block

// bf16 copies of the LoRA factors, plain and scaled by gamma, zero-padded to LORA_PAD.
__global__ void k_lora_cast(int rank, int d_in, int d_out, float gamma, const float* __restrict__ A,
                            const float* __restrict__ B, __nv_bfloat16* __restrict__ Ab,
                            __nv_bfloat16* __restrict__ gAb, __nv_bfloat16* __restrict__ Bb,
                            __nv_bfloat16* __restrict__ gBb) {
  const size_t na = (size_t)LORA_PAD * d_in, nb = (size_t)d_out * LORA_PAD;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < na + nb; e += stride) {
    if (e < na) {
      const int k = (int)(e / d_in);
      const float v = k < rank ? A[e] : 0.f;          // same flat index: A is [rank, d_in]
      Ab[e] = __float2bfloat16_rn(v);
      gAb[e] = __float2bfloat16_rn(gamma * v);
    } else {
      const size_t f = e - na;
      const int o = (int)(f / LORA_PAD), k = (int)(f % LORA_PAD);
      const float v = k < rank ? B[(size_t)o * rank + k] : 0.f;
      Bb[f] = __float2bfloat16_rn(v);
      gBb[f] = __float2bfloat16_rn(gamma * v);
    }
  }
}

// Device scratch of the variant paths (all offsets 256-byte aligned).
struct VariantScratch {
  __nv_bfloat16 *Ab, *gAb, *Bb, *gBb, *Xt, *dYt;
  size_t bytes;
};

inline size_t variant_align(size_t x) { return (x + 255) / 256 * 256; }

inline VariantScratch variant_scratch(const Params& p, void* base) {
  VariantScratch v{};
  unsigned char* c = static_cast<unsigned char*>(base);
  size_t off = 0;
  auto take = [&](size_t n) { unsigned char* q = c ? c + off : nullptr; off += variant_align(n); return q; };
  v.Ab = reinterpret_cast<__nv_bfloat16*>(take((size_t)LORA_PAD * p.d_in * 2));
  v.gAb = reinterpret_cast<__nv_bfloat16*>(take((size_t)LORA_PAD * p.d_in * 2));
  v.Bb = reinterpret_cast<__nv_bfloat16*>(take((size_t)p.d_out * LORA_PAD * 2));
  v.gBb = reinterpret_cast<__nv_bfloat16*>(take((size_t)p.d_out * LORA_PAD * 2));
  v.Xt = reinterpret_cast<__nv_bfloat16*>(take((size_t)p.tokens * LORA_PAD * 2));
  v.dYt = reinterpret_cast<__nv_bfloat16*>(take((size_t)p.tokens * LORA_PAD * 2));
  v.bytes = off;
  return v;
}

inline l4q_status launch_lora_cast(const Params& p, const float* A, const float* B, const VariantScratch& v,
                                   cudaStream_t st) {
  const size_t n = (size_t)LORA_PAD * p.d_in + (size_t)p.d_out * LORA_PAD;
  const int blocks = (int)std::min<size_t>((n + 255) / 256, (size_t)sm_count() * 8);
  k_lora_cast<<<blocks, 256, 0, st>>>(p.rank, p.d_in, p.d_out, p.gamma, A, B, v.Ab, v.gAb, v.Bb, v.gBb);
  return cudaGetLastError() == cudaSuccess ? L4Q_OK : L4Q_ERR_CUDA;
}

// Xt[tokens, 64] = X[tokens, d_in] Ab[64, d_in]^T      (the input of B in Eq. 1)
inline l4q_status gemm_lora_down_bf16(const Params& p, const void* X, const VariantScratch& v, cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!make_tmap_bf16(&ta, X, p.tokens, p.d_in, BM) || !make_tmap_bf16(&tb, v.Ab, LORA_PAD, p.d_in, LORA_PAD))
    return cuda_fail();
  GemmArgs g{};
  g.M = p.tokens; g.N = LORA_PAD; g.K = p.d_in;
  g.C = v.Xt;
  return launch_gemm<false, false, EPI_STORE, 0, 8, 64>(ta, tb, g, st);
}

// dYt[tokens, 64] = dY[tokens, d_out] Bb[d_out, 64]    (the gradient at the output of A)
inline l4q_status gemm_lora_up_t_bf16(const Params& p, const void* dY, const VariantScratch& v, cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!make_tmap_bf16(&ta, dY, p.tokens, p.d_out, BM) || !make_tmap_bf16(&tb, v.Bb, p.d_out, LORA_PAD, BK))
    return cuda_fail();
  GemmArgs g{};
  g.M = p.tokens; g.N = LORA_PAD; g.K = p.d_out;
  g.C = v.dYt;
  return launch_gemm<false, true, EPI_STORE, 0, 8, 64>(ta, tb, g, st);
}

// Y[tokens, d_out] = X W^T + Xt gBb^T                    (Eq. 1; W = W0 or Q(W0))
inline l4q_status gemm_forward_lora_bf16(const Params& p, const void* X, const void* W, const VariantScratch& v,
                                         void* Y, cudaStream_t st) {
  CUtensorMap ta, tb, ta2, tb2;
  if (!make_tmap_bf16(&ta, X, p.tokens, p.d_in, BM) || !make_tmap_bf16(&tb, W, p.d_out, p.d_in, BN) ||
      !make_tmap_bf16(&ta2, v.Xt, p.tokens, LORA_PAD, BM) || !make_tmap_bf16(&tb2, v.gBb, p.d_out, LORA_PAD, BN))
    return cuda_fail();
  GemmArgs g{};
  g.M = p.tokens; g.N = p.d_out; g.K = p.d_in;
  g.num_kb2 = 1;
  g.C = reinterpret_cast<__nv_bfloat16*>(Y);
  return launch_gemm<false, false, EPI_STORE, 0, 4, BN, true>(ta, tb, g, st, &ta2, &tb2);
}

// dX[tokens, d_in] = dY W + dYt gAb
inline l4q_status gemm_dgrad_lora_bf16(const Params& p, const void* dY, const void* W, const VariantScratch& v,
                                       void* dX, cudaStream_t st) {
  CUtensorMap ta, tb, ta2, tb2;
  if (!make_tmap_bf16(&ta, dY, p.tokens, p.d_out, BM) || !make_tmap_bf16(&tb, W, p.d_out, p.d_in, BK) ||
      !make_tmap_bf16(&ta2, v.dYt, p.tokens, LORA_PAD, BM) || !make_tmap_bf16(&tb2, v.gAb, LORA_PAD, p.d_in, BK))
    return cuda_fail();
  GemmArgs g{};
  g.M = p.tokens; g.N = p.d_in; g.K = p.d_out;
  g.num_kb2 = 1;
  g.C = reinterpret_cast<__nv_bfloat16*>(dX);
  return launch_gemm<false, true, EPI_STORE, 0, 4, BN, true>(ta, tb, g, st, &ta2, &tb2);
}

// dA[rank, d_in] += gamma dYt^T X      (Eq. 2; dA zero on entry; cut along the tokens over the idle SMs)
inline l4q_status gemm_lora_da_bf16(const Params& p, const void* X, const VariantScratch& v, float* dA,
                                    cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!make_tmap_bf16(&ta, v.dYt, p.tokens, LORA_PAD, BK) || !make_tmap_bf16(&tb, X, p.tokens, p.d_in, BK))
    return cuda_fail();
  GemmArgs g{};
  g.M = p.rank; g.N = p.d_in; g.K = p.tokens;
  g.C32 = dA; g.ldc = p.d_in; g.scale = p.gamma;
  return launch_gemm<true, true, EPI_ADD_F32, 0, 4, BN>(ta, tb, g, st);
}

// dB[d_out, rank] += gamma dY^T Xt     (Eq. 2; dB zero on entry)
inline l4q_status gemm_lora_db_bf16(const Params& p, const void* dY, const VariantScratch& v, float* dB,
                                    cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!make_tmap_bf16(&ta, dY, p.tokens, p.d_out, BK) || !make_tmap_bf16(&tb, v.Xt, p.tokens, LORA_PAD, BK))
    return cuda_fail();
  GemmArgs g{};
  g.M = p.d_out; g.N = p.rank; g.K = p.tokens;
  g.C32 = dB; g.ldc = p.rank; g.scale = p.gamma;
  return launch_gemm<true, true, EPI_ADD_F32, 0, 8, 64>(ta, tb, g, st);
}

}  // namespace l4q
