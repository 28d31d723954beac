// Shared device/host helpers of the L4Q library: problem parameters, the
// element-wise quantizer arithmetic (Eq. 7-9) and small utilities.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/l4q.h"

namespace l4q {

// Problem parameters in the form the kernels consume.
struct Params {
  int tokens, d_in, d_out, rank, bits, group, ngroups;
  float gamma;        // alpha / rank            (Eq. 7)
  float qn, qp;       // integer grid bounds     (Eq. 3)
  float grad_scale;
};

// Device status word: 0 = ok, otherwise an l4q_status recorded by a kernel
// that gave up on a bounded wait.  Read and cleared by l4q_check().
__device__ unsigned int g_l4q_status;

// Grid coordinate w, code w~ and dequantized value W_q of one merged weight.
//   w  = (W_comb - b) * (1/s)      (App. A.2, definition of w; reciprocal taken once per group)
//   w~ = rint(clamp(w, Q_N, Q_P))  (Eq. 8; rint = round-half-to-even)
//   Wq = w~ * s + b                (Eq. 9)
struct QuantElem {
  float w, code, wq;
};

__device__ __forceinline__ QuantElem quantize_elem(float w_comb, float s, float rs, float b, float qn, float qp) {
  QuantElem q;
  q.w = (w_comb - b) * rs;
  q.code = rintf(fminf(fmaxf(q.w, qn), qp));
  q.wq = fmaf(q.code, s, b);
  return q;
}

// In-range test of the straight-through estimator (App. A.1): Q_N <= w <= Q_P on
// the unrounded w, inclusive, widened by 2^-10 of a quantization step so that an
// element a min/max initialisation puts exactly on a bound counts as inside
// whichever way the last bit of s was rounded (Table 4: zero clipping at init).
constexpr float kMaskGuard = 0.0009765625f;

__device__ __forceinline__ bool ste_in_range(float w, float qn, float qp) {
  return (w >= qn - kMaskGuard) && (w <= qp + kMaskGuard);
}

// What the weight-gradient reduction needs to know about one weight besides G, in one number
// (App. A.1): where the STE passes the gradient (Q_N <= w <= Q_P) it is dW_q/ds = w~ - w, a
// value in [-1/2, 1/2]; where w was clamped it is a sentinel, -2 below Q_N and +2 above Q_P
// (there dW_q/ds = Q_N or Q_P and dW_q/db = 1).  Stored as fp16 between the two kernels of the
// backward pass.
constexpr float kSteBelow = -2.f, kSteAbove = 2.f;

__device__ __forceinline__ float ste_factor(const QuantElem& q, float qn, float qp) {
  if (ste_in_range(q.w, qn, qp)) return q.code - q.w;
  return q.w < qn ? kSteBelow : kSteAbove;
}

// W_comb = W0 + gamma * acc, acc = sum_k B[o,k] A[k,j]      (Eq. 7)
__device__ __forceinline__ float merge_elem(float w0, float acc, float gamma) { return fmaf(gamma, acc, w0); }

__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xFFFF0000u); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Status of a failed runtime call.  Reads the runtime's last-error word so that the failure does not surface a
// second time, as the result of an unrelated later call of the same thread.
inline l4q_status cuda_fail() {
  (void)cudaGetLastError();
  return L4Q_ERR_CUDA;
}

// Layout of the STE factor array that the weight-tile kernel hands to the weight-gradient kernel (internal, in the
// workspace): tiles of 128 rows x 128 columns, each one contiguous block of 32 KB ordered [piece of 8 columns]
// [row][8 values], tiles row-major over (row tile, column tile).  A thread that owns a weight row reads 16 bytes
// per piece, and the 32 rows of a warp are then 512 contiguous bytes; the producer writes a tile as one bulk copy.
constexpr int FACTOR_TILE_ELEMS = 128 * 128;
__host__ __device__ inline int factor_tiles_n(int d_in) { return (d_in + 127) >> 7; }
__host__ __device__ inline size_t factor_index(int o, int col, int tiles_n) {
  return ((((size_t)(o >> 7) * tiles_n + (col >> 7)) * 16 + ((col & 127) >> 3)) * 128 + (o & 127)) * 8 + (col & 7);
}
__host__ __device__ inline size_t factor_elems(int d_out, int d_in) {
  return (size_t)((d_out + 127) >> 7) * factor_tiles_n(d_in) * FACTOR_TILE_ELEMS;
}

}  // namespace l4q
