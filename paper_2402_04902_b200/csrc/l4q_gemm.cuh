// bf16 tensor-core GEMMs of the L4Q layer on sm_100a: one persistent,
// warp-specialised kernel template (TMA -> 128B-swizzled shared memory ->
// tcgen05.mma -> fp32 accumulators in tensor memory -> epilogue warps).
//
//   forward   Y  = X  Wq^T   A = X  (K-major),   B = Wq (K-major),   K = d_in     (Eq. 10)
//   dgrad     dX = dY Wq     A = dY (K-major),   B = Wq (MN-major),  K = d_out
//   wgrad     G  = dY^T X    A = dY (MN-major),  B = X  (MN-major),  K = tokens   (Eq. 11)
//
// The wgrad epilogue never writes G: each 128 x 256 tile of G is reduced from
// tensor memory into ds, db (Eq. 5-6), dA and dB (Eq. 13-14), recomputing the
// quantizer state of the tile's weights from W0, A, B, s, b (App. E.2).
//
// Roles (384 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM
// owner, warps 4..11 = two epilogue groups of 128 threads (each group drains
// half of the tile's columns; a warp reads the TMEM lane quarter warp_id % 4).
// Two accumulator stages of 256 TMEM columns let the epilogue of tile t overlap
// the main loop of tile t + 1.
//
// Every wait is bounded; when one expires the kernel records L4Q_ERR_TIMEOUT in
// the device status word, stops issuing work, lets its copies land and frees
// its tensor memory before returning.
#pragma once

#include <algorithm>

#include "l4q_common.cuh"
#include "l4q_ptx.cuh"

namespace l4q {

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int A_STAGE_BYTES = BM * BK * 2;   // 16 KB
constexpr int B_STAGE_BYTES = BN * BK * 2;   // 32 KB
constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr int GEMM_THREADS = 384;
constexpr int EPI_FIRST_WARP = 4;
constexpr int EPI_GROUPS = 2;
constexpr int EPI_THREADS = EPI_GROUPS * 128;
constexpr int ACC_STAGES = 2;
constexpr int TMEM_COLS = ACC_STAGES * BN;   // 512: all of tensor memory
constexpr int STG_LD = 33;                   // padded row length of the wgrad staging tile
constexpr int STG_BYTES = EPI_GROUPS * 128 * STG_LD * 4;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;   // ~2 s at B200 clocks

enum { EPI_STORE = 0, EPI_WGRAD = 1 };

struct GemmArgs {
  int M, N, K;                 // GEMM extents
  int tiles_m, tiles_n, num_kb;
  // EPI_STORE
  __nv_bfloat16* C;            // [M, N] row-major
  // EPI_WGRAD (M = d_out, N = d_in)
  Params p;
  const __nv_bfloat16* W0;
  const float *A, *B, *s, *b;
  float *dA, *dB, *ds, *db;
};

struct __align__(8) GemmBarriers {
  uint64_t full[8], empty[8];
  uint64_t tmem_full[ACC_STAGES], tmem_empty[ACC_STAGES];
  uint32_t tmem_base;
  volatile uint32_t abort;
};

inline size_t gemm_smem_bytes(int stages, int epi_bytes) {
  return 1024 /*alignment slack*/ + (size_t)stages * STAGE_BYTES + (size_t)epi_bytes + sizeof(GemmBarriers);
}

// Bounded mbarrier wait.  Returns immediately once the CTA's abort flag is set.
__device__ __forceinline__ void bounded_wait(uint64_t* bar, uint32_t parity, GemmBarriers* bars) {
  if (ptx::mbar_try_wait(bar, parity)) return;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!ptx::mbar_try_wait(bar, parity)) {
    if ((++spins & 0xFFu) == 0) {
      if (bars->abort) return;
      if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
        bars->abort = 1;
        atomicExch(&g_l4q_status, (unsigned int)L4Q_ERR_TIMEOUT);
        return;
      }
    }
  }
}

// Tile order: bands of 16 tile-rows; inside a band the row index runs fastest, so
// a wave of ~148 tiles touches ~16 row panels and ~9 column panels (L2 reuse).
__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int& tm, int& tn) {
  constexpr int GROUP = 16;
  const int per_band = GROUP * tiles_n;
  const int band = t / per_band;
  const int first = band * GROUP;
  const int rows = min(GROUP, tiles_m - first);
  const int in_band = t - band * per_band;
  tm = first + in_band % rows;
  tn = in_band / rows;
}

// Shared memory of the wgrad epilogue (after the pipeline stages):
//   stg [2 groups][128 rows][33]  Gm chunk, transposed access for the dA column sums
//   Bs  [128 rows][RANK]          the tile's rows of B (zero beyond d_out)
//   As  [2 groups][RANK][32]      the current 32-column chunk of A, one copy per epilogue group
__host__ __device__ constexpr int wgrad_epi_smem_bytes(int rank) {
  return STG_BYTES + 128 * rank * 4 + EPI_GROUPS * rank * 32 * 4;
}

// Loads this thread's share of A[:, jc : jc+32] (RANK x 32 floats = RANK*8 float4 over 128 threads).
template <int RANK>
__device__ __forceinline__ void load_a_chunk(const GemmArgs& g, int jc, int t, float4 (&regs)[(RANK * 8 + 127) / 128]) {
#pragma unroll
  for (int u = 0; u < (RANK * 8 + 127) / 128; ++u) {
    const int f = t + u * 128;
    const int k = f >> 3, v = f & 7;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    if (f < RANK * 8 && jc + v * 4 < g.p.d_in) a = __ldg(reinterpret_cast<const float4*>(g.A + (size_t)k * g.p.d_in + jc + v * 4));
    regs[u] = a;
  }
}
template <int RANK>
__device__ __forceinline__ void store_a_chunk(float* As_g, int t, const float4 (&regs)[(RANK * 8 + 127) / 128]) {
#pragma unroll
  for (int u = 0; u < (RANK * 8 + 127) / 128; ++u) {
    const int f = t + u * 128;
    if (f < RANK * 8) reinterpret_cast<float4*>(As_g)[f] = regs[u];      // As_g[k][v*4..] with f = k*8 + v
  }
}

// One 128 x 256 tile of G = dY^T X, read from tensor memory and reduced into ds, db, dA, dB.
// Thread = one weight row (TMEM lane) of one epilogue group; the group owns 4 chunks of 32 columns.
// Everything that does not depend on the accumulator (B rows, the first A chunk) is fetched before
// waiting for the MMAs; W0, s, b and the next A chunk are fetched ahead of the arithmetic that
// precedes their use, so that the loads' latency hides behind the FMA loops.
template <int RANK>
__device__ __forceinline__ void wgrad_epilogue_tile(const GemmArgs& g, int m0, int n0, uint32_t tmem_acc, int quarter,
                                                    int lane, int eg, float* epi_smem, GemmBarriers* bars,
                                                    uint64_t* tmem_full_bar, uint32_t full_parity,
                                                    uint64_t* tmem_empty_bar) {
  const Params& p = g.p;
  float* stg_g = epi_smem + (size_t)eg * 128 * STG_LD;
  float* Bs = epi_smem + EPI_GROUPS * 128 * STG_LD;
  float* As_g = Bs + 128 * RANK + (size_t)eg * RANK * 32;
  const int t = quarter * 32 + lane;                   // row in tile = thread index within the group
  const int t256 = eg * 128 + t;
  const int o = m0 + t;
  const bool row_ok = o < p.d_out;
  constexpr int CHUNKS_PER_GROUP = (BN / 32) / EPI_GROUPS;
  constexpr int A_REGS = (RANK * 8 + 127) / 128;

  // ---- before the accumulator is ready ----
  ptx::named_bar_sync(3, EPI_THREADS);                 // both groups are done with the previous tile's Bs
#pragma unroll
  for (int u = 0; u < (32 * RANK + EPI_THREADS - 1) / EPI_THREADS; ++u) {
    const int f = t256 + u * EPI_THREADS;              // float4 index into Bs
    if (f < 32 * RANK) {
      const int row = f / (RANK / 4), kq = f % (RANK / 4);
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (m0 + row < p.d_out) v = __ldg(reinterpret_cast<const float4*>(g.B + (size_t)(m0 + row) * RANK + kq * 4));
      reinterpret_cast<float4*>(Bs)[f] = v;
    }
  }
  {
    float4 a0[A_REGS];
    load_a_chunk<RANK>(g, n0 + eg * CHUNKS_PER_GROUP * 32, t, a0);
    store_a_chunk<RANK>(As_g, t, a0);
  }
  float brow[RANK];
#pragma unroll
  for (int k = 0; k < RANK; k += 4) {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row_ok) v = __ldg(reinterpret_cast<const float4*>(g.B + (size_t)o * RANK + k));
    brow[k] = v.x; brow[k + 1] = v.y; brow[k + 2] = v.z; brow[k + 3] = v.w;
  }
  float dBacc[RANK];
#pragma unroll
  for (int k = 0; k < RANK; ++k) dBacc[k] = 0.f;
  ptx::named_bar_sync(3, EPI_THREADS);                 // Bs and the first A chunk are visible

  bounded_wait(tmem_full_bar, full_parity, bars);
  ptx::tc_fence_after_sync();

  float ds_acc = 0.f, db_acc = 0.f;
  int cur_grp = -1;

#pragma unroll 1
  for (int cc = 0; cc < CHUNKS_PER_GROUP; ++cc) {
    const int c = eg * CHUNKS_PER_GROUP + cc;
    const int jc = n0 + c * 32;                        // first column of the chunk

    // loads issued ahead of their use
    uint4 wraw[4];
    float sv[4], bv[4];
    int grp[4];
#pragma unroll
    for (int sub = 0; sub < 4; ++sub) {
      const int j = jc + sub * 8;
      const bool ok = row_ok && j < p.d_in;
      grp[sub] = ok ? j / p.group : -1;
      wraw[sub] = ok ? __ldg(reinterpret_cast<const uint4*>(g.W0 + (size_t)o * p.d_in + j)) : make_uint4(0, 0, 0, 0);
      sv[sub] = ok ? __ldg(g.s + (size_t)o * p.ngroups + grp[sub]) : 1.f;
      bv[sub] = ok ? __ldg(g.b + (size_t)o * p.ngroups + grp[sub]) : 0.f;
    }
    float4 a_next[A_REGS];
    if (cc + 1 < CHUNKS_PER_GROUP) load_a_chunk<RANK>(g, jc + 32, t, a_next);

    uint32_t raw[32];
    ptx::tmem_ld_32x32(tmem_acc + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * 32), raw);
    ptx::tmem_ld_wait();
    if (cc == CHUNKS_PER_GROUP - 1) {                  // accumulator stage fully read by this thread
      ptx::tc_fence_before_sync();
      ptx::mbar_arrive(tmem_empty_bar);
    }
    float G[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) G[e] = __uint_as_float(raw[e]);

    // merge: acc[e] = sum_k B[o,k] A[k, jc+e]                                  (Eq. 7)
    float acc[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) acc[e] = 0.f;
#pragma unroll
    for (int k = 0; k < RANK; ++k) {
      const float4* arow = reinterpret_cast<const float4*>(As_g + k * 32);
#pragma unroll
      for (int v = 0; v < 8; ++v) {
        const float4 a = arow[v];
        acc[v * 4 + 0] = fmaf(brow[k], a.x, acc[v * 4 + 0]);
        acc[v * 4 + 1] = fmaf(brow[k], a.y, acc[v * 4 + 1]);
        acc[v * 4 + 2] = fmaf(brow[k], a.z, acc[v * 4 + 2]);
        acc[v * 4 + 3] = fmaf(brow[k], a.w, acc[v * 4 + 3]);
      }
    }

    // quantizer state, STE gate, ds / db partial sums                           (Eq. 8, 5, 6)
#pragma unroll
    for (int sub = 0; sub < 4; ++sub) {
      if (grp[sub] >= 0) {
        if (grp[sub] != cur_grp) {
          if (cur_grp >= 0) {
            atomicAdd(&g.ds[(size_t)o * p.ngroups + cur_grp], p.grad_scale * ds_acc);
            atomicAdd(&g.db[(size_t)o * p.ngroups + cur_grp], p.grad_scale * db_acc);
          }
          cur_grp = grp[sub]; ds_acc = 0.f; db_acc = 0.f;
        }
        const float rs = 1.0f / sv[sub];
        const uint4 wr = wraw[sub];
        const float w0[8] = {bf16_lo(wr.x), bf16_hi(wr.x), bf16_lo(wr.y), bf16_hi(wr.y),
                             bf16_lo(wr.z), bf16_hi(wr.z), bf16_lo(wr.w), bf16_hi(wr.w)};
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int idx = sub * 8 + e;
          const QuantElem q = quantize_elem(merge_elem(w0[e], acc[idx], p.gamma), sv[sub], rs, bv[sub], p.qn, p.qp);
          const float Gv = G[idx];
          if (ste_in_range(q.w, p.qn, p.qp)) {
            ds_acc = fmaf(Gv, q.code - q.w, ds_acc);
          } else {
            ds_acc = fmaf(Gv, (q.w < p.qn) ? p.qn : p.qp, ds_acc);
            db_acc += Gv;
            G[idx] = 0.f;                              // G becomes G * m
          }
        }
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) G[sub * 8 + e] = 0.f;
      }
    }

    // dB[o,k] += sum_e Gm[e] A[k, jc+e]                                         (Eq. 14)
#pragma unroll
    for (int k = 0; k < RANK; ++k) {
      const float4* arow = reinterpret_cast<const float4*>(As_g + k * 32);
      float part0 = 0.f, part1 = 0.f;
#pragma unroll
      for (int v = 0; v < 8; v += 2) {
        const float4 a = arow[v], a2 = arow[v + 1];
        part0 = fmaf(G[v * 4 + 0], a.x, part0);
        part0 = fmaf(G[v * 4 + 1], a.y, part0);
        part0 = fmaf(G[v * 4 + 2], a.z, part0);
        part0 = fmaf(G[v * 4 + 3], a.w, part0);
        part1 = fmaf(G[v * 4 + 4], a2.x, part1);
        part1 = fmaf(G[v * 4 + 5], a2.y, part1);
        part1 = fmaf(G[v * 4 + 6], a2.z, part1);
        part1 = fmaf(G[v * 4 + 7], a2.w, part1);
      }
      dBacc[k] += part0 + part1;
    }

    // dA[k, jc+col] += sum_rows B[o,k] Gm[o, col]: transpose through shared memory   (Eq. 13)
#pragma unroll
    for (int e = 0; e < 32; ++e) stg_g[t * STG_LD + e] = G[e];
    ptx::named_bar_sync(1 + eg, 128);                  // Gm chunk visible; everyone is past the reads of As_g
    if (cc + 1 < CHUNKS_PER_GROUP) store_a_chunk<RANK>(As_g, t, a_next);
    {
      const int col = t & 31, rq = t >> 5;
      float acc_a[RANK];
#pragma unroll
      for (int k = 0; k < RANK; ++k) acc_a[k] = 0.f;
#pragma unroll 4
      for (int rr = 0; rr < 32; ++rr) {
        const int r2 = rq * 32 + rr;
        const float gm = stg_g[r2 * STG_LD + col];
        const float4* b4 = reinterpret_cast<const float4*>(Bs + r2 * RANK);
#pragma unroll
        for (int k = 0; k < RANK; k += 4) {
          const float4 bq = b4[k >> 2];
          acc_a[k] = fmaf(bq.x, gm, acc_a[k]);
          acc_a[k + 1] = fmaf(bq.y, gm, acc_a[k + 1]);
          acc_a[k + 2] = fmaf(bq.z, gm, acc_a[k + 2]);
          acc_a[k + 3] = fmaf(bq.w, gm, acc_a[k + 3]);
        }
      }
      const int ja = jc + col;
      if (ja < p.d_in) {
#pragma unroll
        for (int k = 0; k < RANK; ++k) atomicAdd(&g.dA[(size_t)k * p.d_in + ja], p.gamma * acc_a[k]);
      }
    }
    ptx::named_bar_sync(1 + eg, 128);                  // staging tile reusable, next A chunk visible
  }

  if (row_ok) {
    if (cur_grp >= 0) {
      atomicAdd(&g.ds[(size_t)o * p.ngroups + cur_grp], p.grad_scale * ds_acc);
      atomicAdd(&g.db[(size_t)o * p.ngroups + cur_grp], p.grad_scale * db_acc);
    }
#pragma unroll
    for (int k = 0; k < RANK; ++k) atomicAdd(&g.dB[(size_t)o * RANK + k], p.gamma * dBacc[k]);
  }
}

template <bool A_MN, bool B_MN, int EPI, int RANK, int STAGES>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
k_gemm_bf16(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const GemmArgs g) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* stage_base = smem;
  constexpr int EPI_SMEM = (EPI == EPI_WGRAD) ? wgrad_epi_smem_bytes(RANK) : 0;
  float* epi_smem = reinterpret_cast<float*>(smem + (size_t)STAGES * STAGE_BYTES);
  GemmBarriers* bars = reinterpret_cast<GemmBarriers*>(smem + (size_t)STAGES * STAGE_BYTES + EPI_SMEM);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = g.tiles_m * g.tiles_n;

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { ptx::mbar_init(&bars->full[i], 1); ptx::mbar_init(&bars->empty[i], 1); }
    for (int i = 0; i < ACC_STAGES; ++i) {
      ptx::mbar_init(&bars->tmem_full[i], 1);
      ptx::mbar_init(&bars->tmem_empty[i], EPI_THREADS);
    }
    bars->abort = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tmap_a);
    ptx::prefetch_tmap(&tmap_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc(&bars->tmem_base, TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      for (int t = blockIdx.x; t < num_tiles && !bars->abort; t += gridDim.x) {
        int tm, tn;
        tile_coords(t, g.tiles_m, g.tiles_n, tm, tn);
        const int m0 = tm * BM, n0 = tn * BN;
        for (int kb = 0; kb < g.num_kb && !bars->abort; ++kb) {
          bounded_wait(&bars->empty[stage], phase ^ 1, bars);
          if (bars->abort) break;
          uint8_t* sa = stage_base + (size_t)stage * STAGE_BYTES;
          uint8_t* sb = sa + A_STAGE_BYTES;
          ptx::mbar_arrive_expect_tx(&bars->full[stage], STAGE_BYTES);
          const int k0 = kb * BK;
          if constexpr (!A_MN) {
            ptx::tma_load_2d(sa, &tmap_a, &bars->full[stage], k0, m0);
          } else {
#pragma unroll
            for (int h = 0; h < BM / 64; ++h)
              ptx::tma_load_2d(sa + h * (64 * BK * 2), &tmap_a, &bars->full[stage], m0 + h * 64, k0);
          }
          if constexpr (!B_MN) {
            ptx::tma_load_2d(sb, &tmap_b, &bars->full[stage], k0, n0);
          } else {
#pragma unroll
            for (int h = 0; h < BN / 64; ++h)
              ptx::tma_load_2d(sb + h * (64 * BK * 2), &tmap_b, &bars->full[stage], n0 + h * 64, k0);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(BM, BN, A_MN, B_MN);
      // K-major: 8-row groups of 128-byte rows are 1024 B apart; a K step of 16 elements is +32 B.
      // MN-major: 8 k-rows of 128 bytes (64 elements along M/N) are 1024 B apart, 64-element
      // blocks along M/N are one TMA box (BK rows x 128 B) apart; a K step of 16 is two row groups.
      constexpr uint32_t A_LBO = A_MN ? (BK * 128) : 16, A_SBO = 1024, A_KSTEP = A_MN ? 2048 : 32;
      constexpr uint32_t B_LBO = B_MN ? (BK * 128) : 16, B_SBO = 1024, B_KSTEP = B_MN ? 2048 : 32;
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      for (int t = blockIdx.x; t < num_tiles && !bars->abort; t += gridDim.x) {
        bounded_wait(&bars->tmem_empty[acc], acc_phase ^ 1, bars);
        if (bars->abort) break;
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < g.num_kb; ++kb) {
          bounded_wait(&bars->full[stage], phase, bars);
          if (bars->abort) break;
          ptx::tc_fence_after_sync();
          const uint32_t sa = ptx::smem_u32(stage_base + (size_t)stage * STAGE_BYTES);
          const uint32_t sb = sa + A_STAGE_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t da = ptx::make_smem_desc_sw128(sa + k * A_KSTEP, A_LBO, A_SBO);
            const uint64_t db = ptx::make_smem_desc_sw128(sb + k * B_KSTEP, B_LBO, B_SBO);
            ptx::mma_bf16_ss(d_tmem, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          ptx::mma_commit(&bars->empty[stage]);       // smem stage reusable once these MMAs retire
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        ptx::mma_commit(&bars->tmem_full[acc]);       // accumulator complete
        if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1; }
      }
    }
    __syncwarp();
  } else if (warp >= EPI_FIRST_WARP) {
    // ------------------------------ epilogue ----------------------------------
    const int quarter = warp & 3;
    const int eg = (warp - EPI_FIRST_WARP) >> 2;
    int acc = 0; uint32_t acc_phase = 0;
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
      int tm, tn;
      tile_coords(t, g.tiles_m, g.tiles_n, tm, tn);
      const int m0 = tm * BM, n0 = tn * BN;
      const uint32_t tmem_acc = tmem_base + (uint32_t)(acc * BN);
      if constexpr (EPI == EPI_STORE) {
        bounded_wait(&bars->tmem_full[acc], acc_phase, bars);
        ptx::tc_fence_after_sync();
        const int row = m0 + quarter * 32 + lane;
        constexpr int CHUNKS_PER_GROUP = (BN / 32) / EPI_GROUPS;
#pragma unroll 1
        for (int cc = 0; cc < CHUNKS_PER_GROUP; ++cc) {
          const int c = eg * CHUNKS_PER_GROUP + cc;
          uint32_t raw[32];
          ptx::tmem_ld_32x32(tmem_acc + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * 32), raw);
          ptx::tmem_ld_wait();
          if (cc == CHUNKS_PER_GROUP - 1) {
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&bars->tmem_empty[acc]);
          }
          if (row < g.M) {
            __nv_bfloat16* dst = g.C + (size_t)row * g.N + n0 + c * 32;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              if (n0 + c * 32 + v * 8 < g.N) {
                uint4 o4;
                o4.x = pack_bf16x2(__uint_as_float(raw[v * 8 + 0]), __uint_as_float(raw[v * 8 + 1]));
                o4.y = pack_bf16x2(__uint_as_float(raw[v * 8 + 2]), __uint_as_float(raw[v * 8 + 3]));
                o4.z = pack_bf16x2(__uint_as_float(raw[v * 8 + 4]), __uint_as_float(raw[v * 8 + 5]));
                o4.w = pack_bf16x2(__uint_as_float(raw[v * 8 + 6]), __uint_as_float(raw[v * 8 + 7]));
                *reinterpret_cast<uint4*>(dst + v * 8) = o4;
              }
            }
          }
        }
      } else {
        wgrad_epilogue_tile<RANK>(g, m0, n0, tmem_acc, quarter, lane, eg, epi_smem, bars, &bars->tmem_full[acc],
                                  acc_phase, &bars->tmem_empty[acc]);
      }
      if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1; }
    }
  }

  // ------------------------------ teardown ------------------------------------
  if (bars->abort) {
    // give copies that are still in flight time to land before the block's shared memory is released
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------

typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline PFN_encodeTiled get_encode_fn() {
  static PFN_encodeTiled fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<PFN_encodeTiled>(p);
  }
  return fn;
}

// bf16 row-major matrix [rows, cols]; box = [box_rows, 64 columns (128 bytes)], 128-byte swizzle, zero fill.
inline bool make_tmap_bf16(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  PFN_encodeTiled enc = get_encode_fn();
  if (!enc) return false;
  const cuuint64_t gdim[2] = {cols, rows};
  const cuuint64_t gstride[1] = {cols * 2};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline int sm_count() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (n <= 0) n = 148;
  }
  return n;
}

template <bool A_MN, bool B_MN, int EPI, int RANK, int STAGES>
l4q_status launch_gemm(const CUtensorMap& ta, const CUtensorMap& tb, GemmArgs& g, cudaStream_t st) {
  g.tiles_m = ceil_div(g.M, BM);
  g.tiles_n = ceil_div(g.N, BN);
  g.num_kb = ceil_div(g.K, BK);
  auto kern = k_gemm_bf16<A_MN, B_MN, EPI, RANK, STAGES>;
  const size_t smem = gemm_smem_bytes(STAGES, EPI == EPI_WGRAD ? wgrad_epi_smem_bytes(RANK) : 0);
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return L4Q_ERR_CUDA;
  const int grid = std::min(g.tiles_m * g.tiles_n, sm_count());
  kern<<<grid, GEMM_THREADS, smem, st>>>(ta, tb, g);
  return cudaGetLastError() == cudaSuccess ? L4Q_OK : L4Q_ERR_CUDA;
}

// Y[tokens, d_out] = X[tokens, d_in] Wq[d_out, d_in]^T
inline l4q_status gemm_forward_bf16(const Params& p, const void* X, const void* Wq, void* Y, cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!make_tmap_bf16(&ta, X, p.tokens, p.d_in, BM) || !make_tmap_bf16(&tb, Wq, p.d_out, p.d_in, BN))
    return L4Q_ERR_CUDA;
  GemmArgs g{};
  g.M = p.tokens; g.N = p.d_out; g.K = p.d_in;
  g.C = reinterpret_cast<__nv_bfloat16*>(Y);
  return launch_gemm<false, false, EPI_STORE, 0, 4>(ta, tb, g, st);
}

// dX[tokens, d_in] = dY[tokens, d_out] Wq[d_out, d_in]
inline l4q_status gemm_dgrad_bf16(const Params& p, const void* dY, const void* Wq, void* dX, cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!make_tmap_bf16(&ta, dY, p.tokens, p.d_out, BM) || !make_tmap_bf16(&tb, Wq, p.d_out, p.d_in, BK))
    return L4Q_ERR_CUDA;
  GemmArgs g{};
  g.M = p.tokens; g.N = p.d_in; g.K = p.d_out;
  g.C = reinterpret_cast<__nv_bfloat16*>(dX);
  return launch_gemm<false, true, EPI_STORE, 0, 4>(ta, tb, g, st);
}

// G[d_out, d_in] = dY^T X reduced on chip into dA, dB, ds, db (which must be zero on entry).
inline l4q_status gemm_wgrad_bf16(const Params& p, const void* X, const void* dY, const void* W0, const float* A,
                                  const float* B, const float* s, const float* b, float* dA, float* dB, float* ds,
                                  float* db, cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!make_tmap_bf16(&ta, dY, p.tokens, p.d_out, BK) || !make_tmap_bf16(&tb, X, p.tokens, p.d_in, BK))
    return L4Q_ERR_CUDA;
  GemmArgs g{};
  g.M = p.d_out; g.N = p.d_in; g.K = p.tokens;
  g.p = p;
  g.W0 = reinterpret_cast<const __nv_bfloat16*>(W0);
  g.A = A; g.B = B; g.s = s; g.b = b;
  g.dA = dA; g.dB = dB; g.ds = ds; g.db = db;
  switch (p.rank) {
    case 8: return launch_gemm<true, true, EPI_WGRAD, 8, 3>(ta, tb, g, st);
    case 16: return launch_gemm<true, true, EPI_WGRAD, 16, 3>(ta, tb, g, st);
    case 32: return launch_gemm<true, true, EPI_WGRAD, 32, 3>(ta, tb, g, st);
    case 64: return launch_gemm<true, true, EPI_WGRAD, 64, 3>(ta, tb, g, st);
    default: return L4Q_ERR_UNSUPPORTED;
  }
}

}  // namespace l4q
