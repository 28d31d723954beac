// fp32 validation path (io_dtype = L4Q_F32): plain FP32-pipe kernels with no
// tensor cores, used to check the layer's arithmetic at small sizes against the
// fp64 oracle to 1e-4.  Correctness only; not tuned.
#pragma once

#include "l4q_common.cuh"

namespace l4q {

constexpr int VT = 64;        // output tile edge
constexpr int VK = 16;        // k-slab
constexpr int V_THREADS = 256;

// C[m, n] = sum_k A(m, k) * B(k, n) with arbitrary element strides, so that the
// three products of the layer are one kernel:
//   Y  = X  Wq^T : A = X  (M x i),  B(k, n) = Wq[n, k]
//   dX = dY Wq   : A = dY (M x o),  B(k, n) = Wq[k, n]
struct GemmView {
  const float* A; long a_m, a_k;
  const float* B; long b_k, b_n;
  int M, N, K;
};

__device__ __forceinline__ void val_tile_mainloop(const GemmView& g, int m0, int n0, float (&acc)[4][4],
                                                  float (*As)[VT + 1], float (*Bs)[VT + 1]) {
  const int tid = threadIdx.x;
  const int tm = tid / 16, tn = tid % 16;
  for (int k0 = 0; k0 < g.K; k0 += VK) {
    for (int idx = tid; idx < VK * VT; idx += V_THREADS) {
      const int kk = idx / VT, mm = idx % VT;
      const int k = k0 + kk;
      const int m = m0 + mm, n = n0 + mm;
      As[kk][mm] = (k < g.K && m < g.M) ? g.A[m * g.a_m + k * g.a_k] : 0.f;
      Bs[kk][mm] = (k < g.K && n < g.N) ? g.B[k * g.b_k + n * g.b_n] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < VK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[kk][tm * 4 + i]; b[i] = Bs[kk][tn * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
}

__global__ void __launch_bounds__(V_THREADS) k_val_gemm(GemmView g, float* __restrict__ C) {
  __shared__ float As[VK][VT + 1], Bs[VK][VT + 1];
  const int m0 = blockIdx.y * VT, n0 = blockIdx.x * VT;
  float acc[4][4] = {};
  val_tile_mainloop(g, m0, n0, acc, As, Bs);
  const int tm = threadIdx.x / 16, tn = threadIdx.x % 16;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int m = m0 + tm * 4 + i, n = n0 + tn * 4 + j;
      if (m < g.M && n < g.N) C[(size_t)m * g.N + n] = acc[i][j];
    }
}

// Weight-gradient tile G = dY^T X (Eq. 11) for a 64 x 64 block of W, reduced on
// chip into ds, db (Eq. 5-6), dA and dB (Eq. 13-14).  G is never written to
// global memory.  ds, db, dA, dB must be zero on entry (fp32 atomics).
__global__ void __launch_bounds__(V_THREADS)
k_val_wgrad(Params p, const float* __restrict__ X, const float* __restrict__ dY, const float* __restrict__ W0,
            const float* __restrict__ A, const float* __restrict__ B, const float* __restrict__ s,
            const float* __restrict__ b, float* __restrict__ dA, float* __restrict__ dB,
            float* __restrict__ ds, float* __restrict__ db) {
  __shared__ float As[VK][VT + 1], Bs[VK][VT + 1];
  __shared__ float Gs[VT][VT + 1];
  const int o0 = blockIdx.y * VT, j0 = blockIdx.x * VT;
  GemmView g;
  g.A = dY; g.a_m = 1; g.a_k = p.d_out;          // A(m = o, k = t) = dY[t, o]
  g.B = X;  g.b_k = p.d_in; g.b_n = 1;           // B(k = t, n = j) = X[t, j]
  g.M = p.d_out; g.N = p.d_in; g.K = p.tokens;
  float acc[4][4] = {};
  val_tile_mainloop(g, o0, j0, acc, As, Bs);
  const int tid = threadIdx.x;
  {
    const int tm = tid / 16, tn = tid % 16;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) Gs[tm * 4 + i][tn * 4 + j] = acc[i][j];
  }
  __syncthreads();

  // pass 1: thread = (row, 16-column run): recompute w, gate G, accumulate ds/db per group
  {
    const int row = tid / 4, run = tid % 4;
    const int o = o0 + row;
    float ds_acc = 0.f, db_acc = 0.f;
    int cur_grp = -1;
    for (int c = 0; c < 16; ++c) {
      const int jj = run * 16 + c, j = j0 + jj;
      float gm = 0.f;
      if (o < p.d_out && j < p.d_in) {
        const int grp = j / p.group;
        if (grp != cur_grp) {
          if (cur_grp >= 0) {
            atomicAdd(&ds[(size_t)o * p.ngroups + cur_grp], p.grad_scale * ds_acc);
            atomicAdd(&db[(size_t)o * p.ngroups + cur_grp], p.grad_scale * db_acc);
          }
          cur_grp = grp; ds_acc = 0.f; db_acc = 0.f;
        }
        float m_acc = 0.f;
        for (int k = 0; k < p.rank; ++k) m_acc = fmaf(B[(size_t)o * p.rank + k], A[(size_t)k * p.d_in + j], m_acc);
        const float sv = s[(size_t)o * p.ngroups + grp], bv = b[(size_t)o * p.ngroups + grp];
        const QuantElem q = quantize_elem(merge_elem(W0[(size_t)o * p.d_in + j], m_acc, p.gamma), sv, 1.0f / sv, bv,
                                          p.qn, p.qp);
        const float G = Gs[row][jj];
        const bool in_range = ste_in_range(q.w, p.qn, p.qp);
        if (in_range) {
          ds_acc = fmaf(G, q.code - q.w, ds_acc);
          gm = G;
        } else {
          ds_acc = fmaf(G, (q.w < p.qn) ? p.qn : p.qp, ds_acc);
          db_acc += G;
        }
      }
      Gs[row][jj] = gm;
    }
    if (cur_grp >= 0) {
      atomicAdd(&ds[(size_t)o * p.ngroups + cur_grp], p.grad_scale * ds_acc);
      atomicAdd(&db[(size_t)o * p.ngroups + cur_grp], p.grad_scale * db_acc);
    }
  }
  __syncthreads();

  // pass 2: dB[o, k] += gamma * sum_j Gm[o, j] A[k, j]   (thread = row, 16-column run)
  {
    const int row = tid / 4, run = tid % 4;
    const int o = o0 + row;
    if (o < p.d_out) {
      for (int k = 0; k < p.rank; ++k) {
        float acc_b = 0.f;
        for (int c = 0; c < 16; ++c) {
          const int jj = run * 16 + c, j = j0 + jj;
          if (j < p.d_in) acc_b = fmaf(Gs[row][jj], A[(size_t)k * p.d_in + j], acc_b);
        }
        atomicAdd(&dB[(size_t)o * p.rank + k], p.gamma * acc_b);
      }
    }
  }
  // pass 3: dA[k, j] += gamma * sum_o B[o, k] Gm[o, j]   (thread = column, 16-row run)
  {
    const int jj = tid % VT, run = tid / VT;
    const int j = j0 + jj;
    if (j < p.d_in) {
      for (int k = 0; k < p.rank; ++k) {
        float acc_a = 0.f;
        for (int c = 0; c < 16; ++c) {
          const int row = run * 16 + c, o = o0 + row;
          if (o < p.d_out) acc_a = fmaf(B[(size_t)o * p.rank + k], Gs[row][jj], acc_a);
        }
        atomicAdd(&dA[(size_t)k * p.d_in + j], p.gamma * acc_a);
      }
    }
  }
}

}  // namespace l4q
