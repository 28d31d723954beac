// Weight-tile kernel: merge (Eq. 7) + fake-quantize (Eq. 8-9) one 64 x 256 tile
// of the weight per thread block, then either
//   * write the dequantized W_q (bf16 or fp32) for the GEMM kernels, or
//   * bit-pack the unsigned codes and narrow s, b to fp16 (export, Sec. 3.2).
// HBM-bound by design: W0 is read with 128-bit loads, one 8-element vector per
// thread per row, and every output line is written fully coalesced.  The rank-r
// merge runs on the FP32 pipe with an 8-row x 8-column register block per
// thread so that one shared-memory read of A feeds 8 rows.
#pragma once

#include "l4q_common.cuh"

namespace l4q {

constexpr int WT_ROWS = 64;      // rows of W per block
constexpr int WT_COLS = 256;     // columns of W per block
constexpr int WT_THREADS = 256;  // 8 warps; warp w owns rows [8w, 8w+8), lane l columns [8l, 8l+8)

enum { WT_MODE_DEQUANT = 0, WT_MODE_PACK = 1, WT_MODE_ERROR = 2 };

inline size_t weight_tile_smem_bytes(int rank) {
  return (size_t)rank * (WT_COLS + WT_ROWS) * sizeof(float);
}

template <bool IO_BF16>
__device__ __forceinline__ void load_w0_vec8(const void* W0, size_t elem_off, float (&v)[8]) {
  if constexpr (IO_BF16) {
    const uint4 raw = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(W0) + elem_off);
    v[0] = bf16_lo(raw.x); v[1] = bf16_hi(raw.x); v[2] = bf16_lo(raw.y); v[3] = bf16_hi(raw.y);
    v[4] = bf16_lo(raw.z); v[5] = bf16_hi(raw.z); v[6] = bf16_lo(raw.w); v[7] = bf16_hi(raw.w);
  } else {
    const float4* p = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(W0) + elem_off);
    const float4 a = p[0], b = p[1];
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
}

template <bool IO_BF16, int MODE>
__global__ void __launch_bounds__(WT_THREADS)
k_weight_tile(Params p, const void* __restrict__ W0, const float* __restrict__ A, const float* __restrict__ B,
              const float* __restrict__ s, const float* __restrict__ b,
              void* __restrict__ wq_out,                       // MODE_DEQUANT: [d_out, d_in] io dtype
              __half* __restrict__ f_out,                      // MODE_DEQUANT, optional: STE factors [d_out, d_in]
              uint32_t* __restrict__ codes, __half* __restrict__ s16, __half* __restrict__ b16,    // MODE_PACK
              double* __restrict__ err) {            // MODE_ERROR: {E_quant, E_clip}, accumulated
  extern __shared__ __align__(16) float smem_f[];
  const int r = p.rank;
  float4* A_lo = reinterpret_cast<float4*>(smem_f);            // [r][32]: columns 8l .. 8l+3 of lane l
  float4* A_hi = A_lo + (size_t)r * 32;                        // [r][32]: columns 8l+4 .. 8l+7
  float* Bt = reinterpret_cast<float*>(A_hi + (size_t)r * 32); // [r][64]: B[row0 + row][k] at Bt[k*64 + row]

  const int col0 = blockIdx.x * WT_COLS;
  const int row0 = blockIdx.y * WT_ROWS;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  for (int idx = tid; idx < r * 64; idx += WT_THREADS) {
    const int k = idx >> 6, v = idx & 63;
    const int c = col0 + v * 4;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < p.d_in) a = *reinterpret_cast<const float4*>(A + (size_t)k * p.d_in + c);
    ((v & 1) ? A_hi : A_lo)[k * 32 + (v >> 1)] = a;
  }
  for (int idx = tid; idx < r * WT_ROWS; idx += WT_THREADS) {
    const int row = idx / r, k = idx - row * r;
    const int o = row0 + row;
    Bt[k * WT_ROWS + row] = (o < p.d_out) ? B[(size_t)o * r + k] : 0.f;
  }
  __syncthreads();

  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

  for (int k = 0; k < r; ++k) {
    const float4 a0 = A_lo[k * 32 + lane], a1 = A_hi[k * 32 + lane];
    const float4 b0 = *reinterpret_cast<const float4*>(Bt + k * WT_ROWS + warp * 8);
    const float4 b1 = *reinterpret_cast<const float4*>(Bt + k * WT_ROWS + warp * 8 + 4);
    const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
    const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(bv[i], av[j], acc[i][j]);
  }

  [[maybe_unused]] float e_quant = 0.f, e_clip = 0.f;          // MODE_ERROR: this thread's share of the sums
  const int col = col0 + lane * 8;
  const bool col_ok = col < p.d_in;
  const int grp = col_ok ? col / p.group : 0;
  const int row_words = (int)(((int64_t)p.d_in * p.bits) >> 5);

#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int o = row0 + warp * 8 + i;
    if (o >= p.d_out) break;                      // uniform across the warp
    float code[8];
    float sv = 1.f, bvv = 0.f;
    if (col_ok) {
      float w0[8];
      load_w0_vec8<IO_BF16>(W0, (size_t)o * p.d_in + col, w0);
      sv = s[(size_t)o * p.ngroups + grp];
      bvv = b[(size_t)o * p.ngroups + grp];
      const float rs = 1.0f / sv;
      float wq[8], fac[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const QuantElem q = quantize_elem(merge_elem(w0[j], acc[i][j], p.gamma), sv, rs, bvv, p.qn, p.qp);
        code[j] = q.code;
        wq[j] = q.wq;
        fac[j] = ste_factor(q, p.qn, p.qp);
        if constexpr (MODE == WT_MODE_ERROR) {                 // |W_comb - W_q|, and its part outside the range
          const float e = fabsf(merge_elem(w0[j], acc[i][j], p.gamma) - q.wq);
          e_quant += e;
          if (!ste_in_range(q.w, p.qn, p.qp)) e_clip += e;
        }
      }
      if constexpr (MODE == WT_MODE_DEQUANT) {
        if (f_out != nullptr) {
          __half2 h[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) h[j] = __floats2half2_rn(fac[2 * j], fac[2 * j + 1]);
          *reinterpret_cast<uint4*>(f_out + factor_index(o, col, factor_tiles_n(p.d_in))) = *reinterpret_cast<const uint4*>(h);
        }
        if constexpr (IO_BF16) {
          uint4 out;
          out.x = pack_bf16x2(wq[0], wq[1]); out.y = pack_bf16x2(wq[2], wq[3]);
          out.z = pack_bf16x2(wq[4], wq[5]); out.w = pack_bf16x2(wq[6], wq[7]);
          *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(wq_out) + (size_t)o * p.d_in + col) = out;
        } else {
          float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(wq_out) + (size_t)o * p.d_in + col);
          dst[0] = make_float4(wq[0], wq[1], wq[2], wq[3]);
          dst[1] = make_float4(wq[4], wq[5], wq[6], wq[7]);
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) code[j] = p.qn;
    }
    if constexpr (MODE == WT_MODE_PACK) {
      // unsigned codes u = w~ - Q_N, 8 of them per thread, LSB-first
      uint32_t piece = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) piece |= (uint32_t)(int)(code[j] - p.qn) << (j * p.bits);
      uint32_t* row_codes = codes + (size_t)o * row_words;
      if (p.bits == 4) {
        if (col_ok) row_codes[col >> 3] = piece;                       // 32 lanes -> 128 contiguous bytes
      } else {                                                         // bits == 3: 4 lanes x 24 bits -> 3 words
        const uint32_t next = __shfl_down_sync(0xffffffffu, piece, 1);
        const int t = lane & 3;
        const uint32_t word = (piece >> (8 * t)) | (next << (24 - 8 * t));
        const int widx = ((col >> 3) >> 2) * 3 + t;
        if (t < 3 && widx < row_words) row_codes[widx] = word;        // 24 lanes -> 96 contiguous bytes
      }
      if (col_ok && (col % p.group) == 0) {
        s16[(size_t)o * p.ngroups + grp] = __float2half_rn(sv);
        b16[(size_t)o * p.ngroups + grp] = __float2half_rn(fmaf(sv, p.qn, bvv));
      }
    }
  }
  if constexpr (MODE == WT_MODE_ERROR) {
    // warp sums, then one fp64 atomic per warp and sum
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      e_quant += __shfl_down_sync(0xffffffffu, e_quant, off);
      e_clip += __shfl_down_sync(0xffffffffu, e_clip, off);
    }
    if (lane == 0) {
      atomicAdd(&err[0], (double)e_quant);
      atomicAdd(&err[1], (double)e_clip);
    }
  }
}

// Per-group initialisation of the quantization parameters (Sec. 3.3, Eq. 15; App. B): one warp per group,
// lane = one 8-element piece.  Results on the signed grid of Eq. 3 are shifted to the unsigned grid
// (b' = b + s Q_N) when the layer uses that one.  s is floored at 1e-8 (Eq. 3 needs s > 0).
enum { INIT_LSQ_PLUS = 0, INIT_SYMM = 1, INIT_ASYMM = 2, INIT_L4Q = 3 };

template <bool IO_BF16>
__global__ void __launch_bounds__(256)
k_init_params(Params p, int method, bool signed_grid, const void* __restrict__ W, float* __restrict__ s_out,
              float* __restrict__ b_out) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  const long long total = (long long)p.d_out * p.ngroups;
  const int pieces = p.group >> 3;
  const float qn_s = -(float)(1 << (p.bits - 1)), qp_s = (float)((1 << (p.bits - 1)) - 1);
  for (long long gidx = warp0; gidx < total; gidx += nwarps) {
    const long long row = gidx / p.ngroups;
    const int grp = (int)(gidx - row * p.ngroups);
    const size_t base = (size_t)row * p.d_in + (size_t)grp * p.group;
    float lo = INFINITY, hi = -INFINITY, sum = 0.f;
    for (int c = lane; c < pieces; c += 32) {
      float v[8];
      load_w0_vec8<IO_BF16>(W, base + (size_t)c * 8, v);
#pragma unroll
      for (int j = 0; j < 8; ++j) { lo = fminf(lo, v[j]); hi = fmaxf(hi, v[j]); sum += v[j]; }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, off));
      hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, off));
      sum += __shfl_xor_sync(0xffffffffu, sum, off);
    }
    float sc = 0.f, bs = 0.f;
    if (method == INIT_LSQ_PLUS) {
      const float mu = sum / (float)p.group;
      float ss = 0.f;                                  // second pass: sum of squared deviations
      for (int c = lane; c < pieces; c += 32) {
        float v[8];
        load_w0_vec8<IO_BF16>(W, base + (size_t)c * 8, v);
#pragma unroll
        for (int j = 0; j < 8; ++j) ss = fmaf(v[j] - mu, v[j] - mu, ss);
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
      const float sigma = sqrtf(ss / (float)p.group);
      sc = fmaxf(fabsf(mu - 3.f * sigma), fabsf(mu + 3.f * sigma)) / (float)(1 << (p.bits - 1));
    } else if (method == INIT_SYMM) {
      sc = fmaxf(fabsf(lo), fabsf(hi)) / (float)(1 << (p.bits - 1));
    } else if (method == INIT_ASYMM) {
      sc = fmaxf((hi - lo) / (qp_s - qn_s), 1e-8f);
      bs = signed_grid ? lo - sc * qn_s : lo;          // unsigned grid: b' = b + s Q_N = min W exactly
    } else {
      sc = fmaxf(fabsf(lo / qn_s), fabsf(hi / qp_s));
    }
    sc = fmaxf(sc, 1e-8f);
    if (!signed_grid && method != INIT_ASYMM) bs = sc * qn_s;   // b = 0 on the signed grid
    if (lane == 0) { s_out[gidx] = sc; b_out[gidx] = bs; }
  }
}

// The same initialisation for groups of 8, 16, ..., 256 elements (a power of two of 8-element pieces, at most
// one warp wide): the weight is walked as one linear array of pieces, lane = piece, so every load of a warp is 512
// contiguous bytes and four of them are in flight per thread; the lanes of a group reduce with shuffles, and the
// variance of LSQ+ is taken from the values still in registers.
template <bool IO_BF16>
__global__ void __launch_bounds__(256)
k_init_params_vec(Params p, int method, bool signed_grid, int lanes_log2, const void* __restrict__ W,
                  float* __restrict__ s_out, float* __restrict__ b_out) {
  constexpr int U = 4;
  const int lane = threadIdx.x & 31;
  const int lpg = 1 << lanes_log2;                         // lanes (pieces) per group
  const long long total = (long long)p.d_out * p.d_in / 8;  // pieces; a multiple of lpg
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long nthreads = (long long)gridDim.x * blockDim.x;
  const float qn_s = -(float)(1 << (p.bits - 1)), qp_s = (float)((1 << (p.bits - 1)) - 1);
  const float inv_n = 1.f / (float)p.group;
  for (long long w0 = tid - lane; w0 < total; w0 += nthreads * U) {
    float v[U][8];
    bool ok[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const long long q = w0 + (long long)u * nthreads + lane;
      ok[u] = q < total;
      if (ok[u]) load_w0_vec8<IO_BF16>(W, (size_t)q * 8, v[u]);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float lo = INFINITY, hi = -INFINITY, sum = 0.f;
      if (ok[u]) {
#pragma unroll
        for (int j = 0; j < 8; ++j) { lo = fminf(lo, v[u][j]); hi = fmaxf(hi, v[u][j]); sum += v[u][j]; }
      }
      for (int off = lpg >> 1; off > 0; off >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, off));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, off));
        sum += __shfl_xor_sync(0xffffffffu, sum, off);
      }
      float sc = 0.f, bs = 0.f;
      if (method == INIT_LSQ_PLUS) {
        const float mu = sum * inv_n;
        float ss = 0.f;
        if (ok[u]) {
#pragma unroll
          for (int j = 0; j < 8; ++j) ss = fmaf(v[u][j] - mu, v[u][j] - mu, ss);
        }
        for (int off = lpg >> 1; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
        const float sigma = sqrtf(ss * inv_n);
        sc = fmaxf(fabsf(mu - 3.f * sigma), fabsf(mu + 3.f * sigma)) / (float)(1 << (p.bits - 1));
      } else if (method == INIT_SYMM) {
        sc = fmaxf(fabsf(lo), fabsf(hi)) / (float)(1 << (p.bits - 1));
      } else if (method == INIT_ASYMM) {
        sc = fmaxf((hi - lo) / (qp_s - qn_s), 1e-8f);
        bs = signed_grid ? lo - sc * qn_s : lo;
      } else {
        sc = fmaxf(fabsf(lo / qn_s), fabsf(hi / qp_s));
      }
      sc = fmaxf(sc, 1e-8f);
      if (!signed_grid && method != INIT_ASYMM) bs = sc * qn_s;
      const long long q = w0 + (long long)u * nthreads + lane;
      if (ok[u] && (lane & (lpg - 1)) == 0) { s_out[q >> lanes_log2] = sc; b_out[q >> lanes_log2] = bs; }
    }
  }
}

// One AdamW update of a parameter tensor (App. D: AdamW, decoupled weight decay), everything in one pass:
//   p <- p - lr wd p;  m <- b1 m + (1 - b1) g;  v <- b2 v + (1 - b2) g^2;  p <- p - lr (m / c1) / (sqrt(v / c2) + eps)
// with the bias corrections c1 = 1 - b1^t, c2 = 1 - b2^t computed on the host in double precision.
__global__ void __launch_bounds__(256)
k_adamw(float* __restrict__ param, const float* __restrict__ grad, float* __restrict__ m, float* __restrict__ v,
        size_t n, float lr, float beta1, float beta2, float eps, float weight_decay, float inv_c1, float inv_c2) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const float g = grad[i];
    float p = param[i];
    p = fmaf(-lr * weight_decay, p, p);
    const float mi = fmaf(beta1, m[i], (1.f - beta1) * g);
    const float vi = fmaf(beta2, v[i], (1.f - beta2) * g * g);
    m[i] = mi;
    v[i] = vi;
    param[i] = p - lr * (mi * inv_c1) / (sqrtf(vi * inv_c2) + eps);
  }
}

// The same update for several tensors in one launch (the four trainable tensors of a layer -- A, B, s, b -- are
// small: one launch each is bound by the launch, not by memory).  Element e of the concatenation of the tensors
// belongs to the tensor whose [begin, end) holds it; a thread finds it by scanning the (at most 8) ends.
constexpr int ADAMW_MAX_TENSORS = 8;
struct AdamwTable {
  float* param[ADAMW_MAX_TENSORS];
  const float* grad[ADAMW_MAX_TENSORS];
  float* m[ADAMW_MAX_TENSORS];
  float* v[ADAMW_MAX_TENSORS];
  unsigned long long end[ADAMW_MAX_TENSORS];   // running totals of the element counts
  int count;
};

__global__ void __launch_bounds__(256)
k_adamw_multi(const AdamwTable t, float lr, float beta1, float beta2, float eps, float weight_decay, float inv_c1,
              float inv_c2) {
  const unsigned long long total = t.end[t.count - 1];
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  for (unsigned long long e = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
    int k = 0;
#pragma unroll
    for (int j = 0; j < ADAMW_MAX_TENSORS - 1; ++j) k += (j < t.count - 1 && e >= t.end[j]) ? 1 : 0;
    const size_t i = (size_t)(e - (k ? t.end[k - 1] : 0ull));
    const float g = t.grad[k][i];
    float p = t.param[k][i];
    p = fmaf(-lr * weight_decay, p, p);
    const float mi = fmaf(beta1, t.m[k][i], (1.f - beta1) * g);
    const float vi = fmaf(beta2, t.v[k][i], (1.f - beta2) * g * g);
    t.m[k][i] = mi;
    t.v[k][i] = vi;
    t.param[k][i] = p - lr * (mi * inv_c1) / (sqrtf(vi * inv_c2) + eps);
  }
}

}  // namespace l4q
