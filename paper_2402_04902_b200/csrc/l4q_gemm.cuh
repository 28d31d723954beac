// bf16 tensor-core GEMMs of the L4Q layer on sm_100a: one persistent,
// warp-specialised kernel template (TMA -> 128B-swizzled shared memory ->
// tcgen05.mma -> fp32 accumulators in tensor memory -> epilogue warps).
//
//   forward   Y  = X  Wq^T   A = X  (K-major),   B = Wq (K-major),   K = d_in     (Eq. 10)
//   dgrad     dX = dY Wq     A = dY (K-major),   B = Wq (MN-major),  K = d_out
//   wgrad     G  = dY^T X    A = dY (MN-major),  B = X  (MN-major),  K = tokens   (Eq. 11)
//
// The same template also runs the layers L4Q is compared with (Eq. 1-2, Sec. 3.1): a narrow N tile
// (TN = 64) for the rank-side products X A^T and dY B, one extra K block taken from a second pair
// of tensor maps (EXT) that adds the LoRA path gamma (X A^T) B^T to the main product inside the
// accumulator, and an epilogue that adds a scaled fp32 tile into dA / dB (EPI_ADD_F32).
//
// The wgrad epilogue never writes G: each 128 x 256 tile of G is reduced from
// tensor memory into ds, db (Eq. 5-6), dA and dB (Eq. 13-14).  The quantizer
// state of the tile's weights (STE gate and dW_q/ds) is recomputed in the same
// backward call by the weight-tile kernel (App. E.2) and read here as one fp16
// factor per weight; the contractions with the LoRA factors that give dA and dB
// are two more tcgen05 MMAs per 128 columns, fed from a bf16 copy of G * m in
// shared memory.
//
// Roles (384 threads): warp 0 = TMA producer of operand A, warp 2 = TMA producer
// of operand B, warp 1 = MMA issuer and TMEM owner, warps 4..11 = two epilogue groups of 128 threads (each group drains
// half of the tile's columns; a warp reads the TMEM lane quarter warp_id % 4).
// Two accumulator stages of 256 TMEM columns let the epilogue of tile t overlap
// the main loop of tile t + 1.
//
// Every wait is bounded; when one expires the kernel records L4Q_ERR_TIMEOUT in
// the device status word, stops issuing work, lets its copies land and frees
// its tensor memory before returning.
#pragma once

#include <atomic>

#include <algorithm>

#include "l4q_common.cuh"
#include "l4q_ptx.cuh"

namespace l4q {

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int A_STAGE_BYTES = BM * BK * 2;   // 16 KB
constexpr int B_STAGE_BYTES = BN * BK * 2;   // 32 KB
constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
__host__ __device__ constexpr int stage_bytes_for(int tn) { return A_STAGE_BYTES + tn * BK * 2; }
constexpr int GEMM_THREADS = 384;
constexpr int EPI_FIRST_WARP = 4;
constexpr int EPI_GROUPS = 2;
constexpr int EPI_THREADS = EPI_GROUPS * 128;
constexpr int ACC_STAGES = 2;
constexpr int TMEM_COLS = ACC_STAGES * BN;   // 512: all of tensor memory
constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;   // ~2 s at B200 clocks

enum { EPI_STORE = 0, EPI_WGRAD = 1, EPI_ADD_F32 = 2 };

struct GemmArgs {
  int M, N, K;                 // GEMM extents
  int tiles_m, tiles_n, num_kb;
  int band;                    // tile rows per band of the tile order (see tile_coords)
  int num_kb2;                 // EXT: K blocks taken from the second pair of tensor maps, after the first num_kb
  // EPI_STORE
  __nv_bfloat16* C;            // [M, N] row-major
  // EPI_ADD_F32: C32[row * ldc + col] += scale * acc for row < M, col < N (atomic; C32 zero or partial on entry)
  float* C32;
  int ldc;
  float scale;
  // EPI_WGRAD (M = d_out, N = d_in)
  Params p;
  const __half* F;             // STE factors of the weights (ste_factor), in the factor_index layout
  int f_tiles_n;               // column tiles of that layout
  float *dA, *dB, *ds, *db;
};

struct __align__(8) GemmBarriers {
  uint64_t full[8], empty[8];
  uint64_t tmem_full[ACC_STAGES], tmem_empty[ACC_STAGES];
  uint64_t epi_mma;            // wgrad: the epilogue's own MMAs have completed
  uint64_t epi_ops;            // wgrad: the tile's bf16 slices of A and B^T have landed
  uint32_t tmem_base;
  volatile uint32_t abort;
};

inline size_t gemm_smem_bytes(int stages, int epi_bytes, int stage_bytes = STAGE_BYTES) {
  return 1024 /*alignment slack*/ + (size_t)stages * stage_bytes + (size_t)epi_bytes + sizeof(GemmBarriers);
}

// Bounded mbarrier wait.  Returns true once the phase has completed; false when it gave up because the time limit
// ran out (it then sets the CTA's abort flag and the device status word) or because the abort flag was already set.
template <class Barriers>
__device__ __forceinline__ bool bounded_wait(uint64_t* bar, uint32_t parity, Barriers* bars,
                                             long long limit_cycles = WAIT_LIMIT_CYCLES) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!ptx::mbar_try_wait(bar, parity)) {
    if ((++spins & 0xFFu) == 0) {
      if (bars->abort) return false;
      if (clock64() - t0 > limit_cycles) {
        bars->abort = 1;
        atomicExch(&g_l4q_status, (unsigned int)L4Q_ERR_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

// The same wait for a role that runs ahead of its ring and has time to spare (a TMA producer waiting for a free
// slot, an epilogue warp waiting for a whole tile): between polls the thread sleeps, so that its polling does
// not take issue slots from the warps that share its scheduler.
template <class Barriers>
__device__ __forceinline__ bool bounded_wait_relaxed(uint64_t* bar, uint32_t parity, Barriers* bars, unsigned sleep_ns = 256,
                                                     long long limit_cycles = WAIT_LIMIT_CYCLES) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!ptx::mbar_try_wait(bar, parity)) {
    __nanosleep(sleep_ns);
    if ((++spins & 0x3Fu) == 0) {
      if (bars->abort) return false;
      if (clock64() - t0 > limit_cycles) {
        bars->abort = 1;
        atomicExch(&g_l4q_status, (unsigned int)L4Q_ERR_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

// The same wait on a shared-window address (no generic-to-shared conversion per call).
template <class Barriers>
__device__ __forceinline__ bool bounded_wait_a(uint32_t bar_a, uint32_t parity, Barriers* bars,
                                               long long limit_cycles = WAIT_LIMIT_CYCLES) {
  if (ptx::mbar_try_wait_a(bar_a, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!ptx::mbar_try_wait_a(bar_a, parity)) {
    if ((++spins & 0xFFu) == 0) {
      if (bars->abort) return false;
      if (clock64() - t0 > limit_cycles) {
        bars->abort = 1;
        atomicExch(&g_l4q_status, (unsigned int)L4Q_ERR_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

// Self-test of the error path of bounded_wait: one block waits on a barrier that nothing ever arrives on, with
// a limit of about a millisecond.  The wait gives up, records L4Q_ERR_TIMEOUT and the kernel returns normally.
struct SelftestBarriers { uint64_t never; volatile uint32_t abort; };

__global__ void k_selftest_timeout() {
  __shared__ SelftestBarriers bars;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bars.never, 1);
    bars.abort = 0;
    ptx::fence_mbar_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) bounded_wait(&bars.never, 0, &bars, 2000000LL);
}

// Tile order: bands of `GROUP` tile-rows; inside a band the row index runs fastest, so a wave of ~148 tiles
// touches GROUP row panels and ~148 / GROUP column panels.  The A panels of a band stay in L2 while the B
// panels stream past once per band, so the band is made as tall as L2 allows (tile_band_rows).
__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int GROUP, int& tm, int& tn) {
  const int per_band = GROUP * tiles_n;
  const int band = t / per_band;
  const int first = band * GROUP;
  const int rows = min(GROUP, tiles_m - first);
  const int in_band = t - band * per_band;
  tm = first + in_band % rows;
  tn = in_band / rows;
}

// Work distribution over the persistent CTAs: tile t goes to CTA t mod gridDim.x, so the CTAs of a
// wave work on neighbouring tiles and share operand panels in L2.  With TAIL_SPLIT (wgrad) the tiles
// of the last, partial wave are additionally cut along K into `split` slices, one per otherwise idle
// CTA: the reductions of the wgrad epilogue are linear in G and accumulate with atomics, so a partial
// sum over tokens is just one more contribution.
struct WorkUnit { int tile, kb0, kb1; };

__host__ __device__ inline int tail_split_factor(int tiles, int grid, int num_kb) {
  const int tail = tiles % grid;
  if (tail == 0) return 1;
  const int split = grid / tail;
  return split < 1 ? 1 : (split > num_kb ? num_kb : split);
}

template <bool TAIL_SPLIT>
struct WorkIter {
  int next_tile, num_tiles, num_kb, first_tail, tail, split;
  bool tail_done;
  __device__ WorkIter(int tiles, int kblocks) : next_tile(blockIdx.x), num_tiles(tiles), num_kb(kblocks) {
    const int grid = gridDim.x;
    first_tail = TAIL_SPLIT ? (tiles / grid) * grid : tiles;
    tail = tiles - first_tail;
    split = TAIL_SPLIT ? tail_split_factor(tiles, grid, kblocks) : 1;
    tail_done = false;
  }
  __device__ bool next(WorkUnit& u) {
    if (next_tile < first_tail) {
      u.tile = next_tile; u.kb0 = 0; u.kb1 = num_kb;
      next_tile += gridDim.x;
      return true;
    }
    if (tail_done || (int)blockIdx.x >= tail * split) return false;
    tail_done = true;
    const int slice = blockIdx.x / tail;
    u.tile = first_tail + blockIdx.x % tail;
    u.kb0 = (int)((long long)num_kb * slice / split);
    u.kb1 = (int)((long long)num_kb * (slice + 1) / split);
    return u.kb1 > u.kb0;
  }
};

// Shared memory of the wgrad epilogue (after the pipeline stages; every piece starts on a 1 KB boundary):
//   gm    32 KB            Gm = G * m for 128 columns, bf16, as two 128-row x 64-column tiles in the
//                          128-byte-swizzled layout TMA would produce.  Read by the tensor cores twice:
//                          K-major (rows = weight rows, K = columns) for dB, MN-major (the same bytes,
//                          M = columns, K = weight rows) for dA.
//   abf   4 x RN x 128 B   bf16 copy of A[:, n0 : n0+256], four K-major tiles of 64 columns
//   btbf  2 x RN x 128 B   bf16 copy of B[m0 : m0+128, :]^T, two K-major tiles of 64 weight rows
// RN = max(rank, 16) rows (the MMA's N), rows beyond the rank are zero.
// Up to rank 16 the epilogue works on 64 columns at a time (Gm is one 128 x 64 tile, 16 KB): that leaves room
// for a fourth pipeline stage, which the main loop needs more than the epilogue needs wide steps.
constexpr int GM_BYTES = 128 * 128 * 2;
__host__ __device__ constexpr int wgrad_rn(int rank) { return rank < 16 ? 16 : rank; }
__host__ __device__ constexpr bool wgrad_quarters(int rank) { return wgrad_rn(rank) == 16; }
__host__ __device__ constexpr int wgrad_gm_bytes(int rank) { return wgrad_quarters(rank) ? GM_BYTES / 2 : GM_BYTES; }
__host__ __device__ constexpr int wgrad_epi_smem_bytes(int rank) {
  return wgrad_gm_bytes(rank) + 6 * wgrad_rn(rank) * 128;
}
__host__ __device__ constexpr int wgrad_stages(int rank) { return wgrad_quarters(rank) ? 4 : 3; }
constexpr int STORE_BOX_BYTES = 128 * 64 * 2;       // one staging box of the store epilogue: 128 rows x 64 columns bf16
__host__ __device__ constexpr int store_epi_smem_bytes() { return EPI_GROUPS * STORE_BOX_BYTES; }

template <int N>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t (&r)[N]) {
  static_assert(N == 8 || N == 16 || N == 32, "tcgen05.ld width");
  if constexpr (N == 8) ptx::tmem_ld_32x8(taddr, r);
  else if constexpr (N == 16) ptx::tmem_ld_32x16(taddr, r);
  else ptx::tmem_ld_32x32(taddr, r);
}

// One 128 x 256 tile of G = dY^T X (Eq. 11), read from tensor memory and reduced into ds, db, dA, dB.
//
// The quantizer state of the tile's weights comes from the factor array F that the weight-tile kernel
// of the same backward call wrote (ste_factor): F = w~ - w where the STE passes the gradient, a
// sentinel where w was clamped.  Per element (thread = one weight row = one TMEM lane):
//     ds += G * {Q_N | w~ - w | Q_P}      db += G * (1 - m)      Gm = G * m          (Eq. 5, 6, App. A.1)
// Gm goes to shared memory as bf16 and the two contractions with the LoRA factors run on the tensor
// cores (Eq. 13-14), 128 columns at a time, into accumulator columns this tile has already drained:
//     dB[128 rows, r]   += Gm[128, 128] A[:, cols]^T          (K-major Gm)
//     dA^T[128 cols, r]  = Gm^T[128 cols, 128 rows] B[rows, :] (MN-major view of the same Gm)
// Their results are read back once per tile and added to dA / dB with fp32 atomics; the accumulator
// stage is handed back to the main loop only after that.
template <int RANK>
__device__ __forceinline__ void wgrad_epilogue_tile(const GemmArgs& g, int m0, int n0, uint32_t tmem_acc, int quarter,
                                                    int lane, int eg, uint8_t* epi_smem, GemmBarriers* bars,
                                                    uint64_t* tmem_full_bar, uint32_t full_parity,
                                                    uint64_t* tmem_empty_bar, uint32_t& epi_phase,
                                                    const CUtensorMap* tmap_a16, const CUtensorMap* tmap_bt16,
                                                    uint32_t& ops_phase) {
  constexpr int RN = wgrad_rn(RANK);
  const Params& p = g.p;
  uint8_t* gm = epi_smem;
  uint8_t* abf = gm + GM_BYTES;
  uint8_t* btbf = abf + 4 * RN * 128;
  const int t = quarter * 32 + lane;                   // row in tile = TMEM lane = thread index within the group
  const int t256 = eg * 128 + t;
  const int o = m0 + t;
  const bool row_ok = o < p.d_out;
  const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
  constexpr uint32_t DB_COL = 0, DA_COL0 = RN, DA_COL1 = 128;   // result columns inside the drained accumulator

  // ---- the tile's slices of A and B^T, ready-made bf16 (the operand-split launch of the same backward call wrote
  //      them), by TMA into the swizzled K-major layout the MMAs read.  The MMAs of the previous tile that read
  //      these buffers have completed: every thread waited for them. ----
  if (t256 == 0) {
    ptx::mbar_arrive_expect_tx(&bars->epi_ops, 6 * RN * 128);
#pragma unroll
    for (int blk = 0; blk < 4; ++blk) ptx::tma_load_2d(abf + blk * (RN * 128), tmap_a16, &bars->epi_ops, n0 + blk * 64, 0);
#pragma unroll
    for (int blk = 0; blk < 2; ++blk) ptx::tma_load_2d(btbf + blk * (RN * 128), tmap_bt16, &bars->epi_ops, m0 + blk * 64, 0);
  }

  bounded_wait(tmem_full_bar, full_parity, bars);
  ptx::tc_fence_after_sync();

  float ds_acc = 0.f, db_acc = 0.f;
  int cur_grp = -1;

#pragma unroll 1
  for (int h = 0; h < 2; ++h) {                        // 128 columns at a time; a group owns 64 of them
#pragma unroll 1
    for (int cc = 0; cc < 2; ++cc) {
      const int c = h * 4 + eg * 2 + cc;               // 32-column chunk of the tile
      const int jc = n0 + c * 32;
      uint4 fr[4];
      int grp[4];
#pragma unroll
      for (int sub = 0; sub < 4; ++sub) {
        const int j = jc + sub * 8;
        const bool ok = row_ok && j < p.d_in;
        grp[sub] = ok ? j / p.group : -1;
        fr[sub] = ok ? __ldg(reinterpret_cast<const uint4*>(g.F + factor_index(o, j, g.f_tiles_n))) : make_uint4(0u, 0u, 0u, 0u);
      }
      uint32_t raw[32];
      ptx::tmem_ld_32x32(tmem_acc + lane_base + (uint32_t)(c * 32), raw);
      ptx::tmem_ld_wait();
      float G[32];
#pragma unroll
      for (int e = 0; e < 32; ++e) G[e] = __uint_as_float(raw[e]);

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
          const __half2* fh = reinterpret_cast<const __half2*>(&fr[sub]);
#pragma unroll
          for (int e2 = 0; e2 < 4; ++e2) {
            const float2 f2 = __half22float2(fh[e2]);
            const float fe[2] = {f2.x, f2.y};
#pragma unroll
            for (int e1 = 0; e1 < 2; ++e1) {
              const int idx = sub * 8 + e2 * 2 + e1;
              const float f = fe[e1], Gv = G[idx];
              const bool inr = fabsf(f) < 1.f;           // STE gate m
              ds_acc = fmaf(Gv, inr ? f : (f < 0.f ? p.qn : p.qp), ds_acc);
              db_acc += inr ? 0.f : Gv;
              G[idx] = inr ? Gv : 0.f;                   // G becomes G * m
            }
          }
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) G[sub * 8 + e] = 0.f;
        }
      }
      // Gm chunk -> shared memory: row t, 16-byte pieces (c & 1) * 4 + v of the 64-column tile (c & 3) >> 1
      uint8_t* grow = gm + ((c & 3) >> 1) * (GM_BYTES / 2) + t * 128;
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        uint4 o4;
        o4.x = pack_bf16x2(G[v * 8 + 0], G[v * 8 + 1]); o4.y = pack_bf16x2(G[v * 8 + 2], G[v * 8 + 3]);
        o4.z = pack_bf16x2(G[v * 8 + 4], G[v * 8 + 5]); o4.w = pack_bf16x2(G[v * 8 + 6], G[v * 8 + 7]);
        *reinterpret_cast<uint4*>(grow + ((((c & 1) * 4 + v) ^ (t & 7)) << 4)) = o4;
      }
    }
    ptx::fence_proxy_async_smem();                     // Gm visible to the tensor cores
    ptx::tc_fence_before_sync();                       // the TMEM reads above come before the MMAs below
    ptx::named_bar_sync(3, EPI_THREADS);
    if (t256 == 0 && !bars->abort) {
      if (h == 0) { bounded_wait(&bars->epi_ops, ops_phase, bars); ops_phase ^= 1; }   // the slices of A and B^T
      ptx::tc_fence_after_sync();
      constexpr uint32_t idesc_db = ptx::make_idesc_bf16(128, RN, false, false);
      constexpr uint32_t idesc_da = ptx::make_idesc_bf16(128, RN, true, false);
      const uint32_t gm_a = ptx::smem_u32(gm), abf_a = ptx::smem_u32(abf), bt_a = ptx::smem_u32(btbf);
#pragma unroll
      for (int sb = 0; sb < 2; ++sb) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint64_t da = ptx::make_smem_desc_sw128(gm_a + sb * (GM_BYTES / 2) + k * 32, 16, 1024);
          const uint64_t db = ptx::make_smem_desc_sw128(abf_a + (h * 2 + sb) * (RN * 128) + k * 32, 16, 1024);
          ptx::mma_bf16_ss(tmem_acc + DB_COL, da, db, idesc_db, (h | sb | k) != 0 ? 1u : 0u);
        }
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const uint64_t da = ptx::make_smem_desc_sw128(gm_a + k * 2048, GM_BYTES / 2, 1024);
        const uint64_t db = ptx::make_smem_desc_sw128(bt_a + (k >> 2) * (RN * 128) + (k & 3) * 32, 16, 1024);
        ptx::mma_bf16_ss(tmem_acc + (h == 0 ? DA_COL0 : DA_COL1), da, db, idesc_da, k != 0 ? 1u : 0u);
      }
      ptx::mma_commit(&bars->epi_mma);
    }
    bounded_wait(&bars->epi_mma, epi_phase, bars);     // Gm reusable; after the second half, results complete
    epi_phase ^= 1;
    ptx::tc_fence_after_sync();
  }

  if (row_ok && cur_grp >= 0) {
    atomicAdd(&g.ds[(size_t)o * p.ngroups + cur_grp], p.grad_scale * ds_acc);
    atomicAdd(&g.db[(size_t)o * p.ngroups + cur_grp], p.grad_scale * db_acc);
  }
  {  // dB: lane = weight row; group eg takes half of the ranks
    constexpr int NB = RN / 2;
    uint32_t r[NB];
    tmem_ld_cols<NB>(tmem_acc + lane_base + DB_COL + (uint32_t)(eg * NB), r);
    ptx::tmem_ld_wait();
    if (row_ok) {
#pragma unroll
      for (int k = 0; k < NB; ++k)
        if (eg * NB + k < RANK) atomicAdd(&g.dB[(size_t)o * RANK + eg * NB + k], p.gamma * __uint_as_float(r[k]));
    }
  }
  {  // dA: lane = column of the half eg
    const int col = n0 + eg * 128 + t;
    constexpr int W = RN < 32 ? RN : 32;
#pragma unroll
    for (int kb = 0; kb < RN; kb += W) {
      uint32_t r[W];
      tmem_ld_cols<W>(tmem_acc + lane_base + (eg == 0 ? DA_COL0 : DA_COL1) + (uint32_t)kb, r);
      ptx::tmem_ld_wait();
      if (col < p.d_in) {
#pragma unroll
        for (int k = 0; k < W; ++k)
          if (kb + k < RANK) atomicAdd(&g.dA[(size_t)(kb + k) * p.d_in + col], p.gamma * __uint_as_float(r[k]));
      }
    }
  }
  ptx::tc_fence_before_sync();
  ptx::mbar_arrive(tmem_empty_bar);                    // accumulator stage (and its result columns) free
}

// The same reduction for ranks up to 16, 64 columns at a time (see wgrad_quarters).  Per quarter q the two
// groups drain one 32-column chunk each into a 128 x 64 Gm tile; then
//     dB[128 rows, r]   += Gm[128, 64] A[:, 64 cols]^T           M = 128, K-major Gm
//     dA_q^T[64 cols, r] = Gm^T[64 cols, 128 rows] B[rows, :]    M = 64, MN-major view of the same bytes
// An M = 64 accumulator keeps row j in TMEM lane 32 (j / 16) + j % 16, i.e. 16 rows in the lower half of each
// warp's lane quarter.  Result columns inside the drained accumulator: dB at 0, dA_q at RN (1 + q); after
// quarter q columns [0, 64 (q + 1)) have been read, and RN (2 + q) <= 64 (q + 1) for RN = 16.
template <int RANK>
__device__ __forceinline__ void wgrad_epilogue_tile_q(const GemmArgs& g, int m0, int n0, uint32_t tmem_acc, int quarter,
                                                      int lane, int eg, uint8_t* epi_smem, GemmBarriers* bars,
                                                      uint64_t* tmem_full_bar, uint32_t full_parity,
                                                      uint64_t* tmem_empty_bar, uint32_t& epi_phase,
                                                      const CUtensorMap* tmap_a16, const CUtensorMap* tmap_bt16,
                                                      uint32_t& ops_phase) {
  constexpr int RN = wgrad_rn(RANK);
  static_assert(RN == 16, "quarter path");
  constexpr int GMQ = GM_BYTES / 2;
  const Params& p = g.p;
  uint8_t* gm = epi_smem;
  uint8_t* abf = gm + GMQ;
  uint8_t* btbf = abf + 4 * RN * 128;
  const int t = quarter * 32 + lane;
  const int t256 = eg * 128 + t;
  const int o = m0 + t;
  const bool row_ok = o < p.d_out;
  const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;

  // ---- the tile's bf16 slices of A and B^T by TMA (as in wgrad_epilogue_tile) ----
  if (t256 == 0) {
    ptx::mbar_arrive_expect_tx(&bars->epi_ops, 6 * RN * 128);
#pragma unroll
    for (int blk = 0; blk < 4; ++blk) ptx::tma_load_2d(abf + blk * (RN * 128), tmap_a16, &bars->epi_ops, n0 + blk * 64, 0);
#pragma unroll
    for (int blk = 0; blk < 2; ++blk) ptx::tma_load_2d(btbf + blk * (RN * 128), tmap_bt16, &bars->epi_ops, m0 + blk * 64, 0);
  }

  bounded_wait(tmem_full_bar, full_parity, bars);
  ptx::tc_fence_after_sync();

  float ds_acc = 0.f, db_acc = 0.f;
  int cur_grp = -1;

#pragma unroll 1
  for (int q = 0; q < 4; ++q) {
    const int c = q * 2 + eg;                          // 32-column chunk of the tile
    const int jc = n0 + c * 32;
    uint4 fr[4];
    int grp[4];
#pragma unroll
    for (int sub = 0; sub < 4; ++sub) {
      const int j = jc + sub * 8;
      const bool ok = row_ok && j < p.d_in;
      grp[sub] = ok ? j / p.group : -1;
      fr[sub] = ok ? __ldg(reinterpret_cast<const uint4*>(g.F + factor_index(o, j, g.f_tiles_n))) : make_uint4(0u, 0u, 0u, 0u);
    }
    uint32_t raw[32];
    ptx::tmem_ld_32x32(tmem_acc + lane_base + (uint32_t)(c * 32), raw);
    ptx::tmem_ld_wait();
    float G[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) G[e] = __uint_as_float(raw[e]);
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
        const __half2* fh = reinterpret_cast<const __half2*>(&fr[sub]);
#pragma unroll
        for (int e2 = 0; e2 < 4; ++e2) {
          const float2 f2 = __half22float2(fh[e2]);
          const float fe[2] = {f2.x, f2.y};
#pragma unroll
          for (int e1 = 0; e1 < 2; ++e1) {
            const int idx = sub * 8 + e2 * 2 + e1;
            const float f = fe[e1], Gv = G[idx];
            const bool inr = fabsf(f) < 1.f;           // STE gate m
            ds_acc = fmaf(Gv, inr ? f : (f < 0.f ? p.qn : p.qp), ds_acc);
            db_acc += inr ? 0.f : Gv;
            G[idx] = inr ? Gv : 0.f;
          }
        }
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) G[sub * 8 + e] = 0.f;
      }
    }
    // Gm chunk -> shared memory: row t, 16-byte pieces eg * 4 + v of the quarter's 64-column tile
    uint8_t* grow = gm + t * 128;
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      uint4 o4;
      o4.x = pack_bf16x2(G[v * 8 + 0], G[v * 8 + 1]); o4.y = pack_bf16x2(G[v * 8 + 2], G[v * 8 + 3]);
      o4.z = pack_bf16x2(G[v * 8 + 4], G[v * 8 + 5]); o4.w = pack_bf16x2(G[v * 8 + 6], G[v * 8 + 7]);
      *reinterpret_cast<uint4*>(grow + (((eg * 4 + v) ^ (t & 7)) << 4)) = o4;
    }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    ptx::named_bar_sync(3, EPI_THREADS);
    if (t256 == 0 && !bars->abort) {
      if (q == 0) { bounded_wait(&bars->epi_ops, ops_phase, bars); ops_phase ^= 1; }   // the slices of A and B^T
      ptx::tc_fence_after_sync();
      constexpr uint32_t idesc_db = ptx::make_idesc_bf16(128, RN, false, false);
      constexpr uint32_t idesc_da = ptx::make_idesc_bf16(64, RN, true, false);
      const uint32_t gm_a = ptx::smem_u32(gm), abf_a = ptx::smem_u32(abf), bt_a = ptx::smem_u32(btbf);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint64_t da = ptx::make_smem_desc_sw128(gm_a + k * 32, 16, 1024);
        const uint64_t db = ptx::make_smem_desc_sw128(abf_a + q * (RN * 128) + k * 32, 16, 1024);
        ptx::mma_bf16_ss(tmem_acc, da, db, idesc_db, (q | k) != 0 ? 1u : 0u);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const uint64_t da = ptx::make_smem_desc_sw128(gm_a + k * 2048, GMQ, 1024);   // one 64-column block: LBO unused
        const uint64_t db = ptx::make_smem_desc_sw128(bt_a + (k >> 2) * (RN * 128) + (k & 3) * 32, 16, 1024);
        ptx::mma_bf16_ss(tmem_acc + (uint32_t)(RN * (1 + q)), da, db, idesc_da, k != 0 ? 1u : 0u);
      }
      ptx::mma_commit(&bars->epi_mma);
    }
    bounded_wait(&bars->epi_mma, epi_phase, bars);     // Gm reusable; after the last quarter, results complete
    epi_phase ^= 1;
    ptx::tc_fence_after_sync();
  }

  if (row_ok && cur_grp >= 0) {
    atomicAdd(&g.ds[(size_t)o * p.ngroups + cur_grp], p.grad_scale * ds_acc);
    atomicAdd(&g.db[(size_t)o * p.ngroups + cur_grp], p.grad_scale * db_acc);
  }
  {  // dB: lane = weight row; group eg takes half of the ranks
    constexpr int NB = RN / 2;
    uint32_t r[NB];
    tmem_ld_cols<NB>(tmem_acc + lane_base + (uint32_t)(eg * NB), r);
    ptx::tmem_ld_wait();
    if (row_ok) {
#pragma unroll
      for (int k = 0; k < NB; ++k)
        if (eg * NB + k < RANK) atomicAdd(&g.dB[(size_t)o * RANK + eg * NB + k], p.gamma * __uint_as_float(r[k]));
    }
  }
#pragma unroll
  for (int qq = 0; qq < 2; ++qq) {  // dA: group eg takes quarters 2 eg and 2 eg + 1; lanes 0..15 of a warp hold 16 columns
    const int q = eg * 2 + qq;
    uint32_t r[RN];
    tmem_ld_cols<RN>(tmem_acc + lane_base + (uint32_t)(RN * (1 + q)), r);
    ptx::tmem_ld_wait();
    const int col = n0 + q * 64 + quarter * 16 + lane;
    if (lane < 16 && col < p.d_in) {
#pragma unroll
      for (int k = 0; k < RN; ++k)
        if (k < RANK) atomicAdd(&g.dA[(size_t)k * p.d_in + col], p.gamma * __uint_as_float(r[k]));
    }
  }
  ptx::tc_fence_before_sync();
  ptx::mbar_arrive(tmem_empty_bar);
}

template <bool A_MN, bool B_MN, int EPI, int RANK, int STAGES, int TN = BN, bool EXT = false>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
k_gemm_bf16(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
            const __grid_constant__ CUtensorMap tmap_a2, const __grid_constant__ CUtensorMap tmap_b2,
            const __grid_constant__ CUtensorMap tmap_c, const GemmArgs g) {
  static_assert(TN == 64 || TN == BN, "tile width");
  static_assert(EPI != EPI_WGRAD || (TN == BN && !EXT), "the weight-gradient epilogue works on 256-column tiles");
  constexpr int STAGE_BYTES = stage_bytes_for(TN);           // shadows the 256-column figure
  constexpr int TMEM_COLS = ACC_STAGES * TN;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* stage_base = smem;
  // EPI_STORE on 256-column tiles leaves through shared memory and TMA stores: one 128 x 64 staging box per
  // epilogue group.  (Stores from registers, one weight row per thread, touch 32 lines per instruction and cost
  // the forward GEMM an eighth of its time.)
  constexpr bool TMA_STORE = (EPI == EPI_STORE && TN == BN);
  constexpr int EPI_SMEM = (EPI == EPI_WGRAD) ? wgrad_epi_smem_bytes(RANK) : TMA_STORE ? store_epi_smem_bytes() : 0;
  uint8_t* epi_smem = smem + (size_t)STAGES * STAGE_BYTES;
  GemmBarriers* bars = reinterpret_cast<GemmBarriers*>(smem + (size_t)STAGES * STAGE_BYTES + EPI_SMEM);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = g.tiles_m * g.tiles_n;
  constexpr bool TAIL_SPLIT = (EPI != EPI_STORE);            // reductions with atomics may be cut along K
  const int total_kb = g.num_kb + (EXT ? g.num_kb2 : 0);

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { ptx::mbar_init(&bars->full[i], 1); ptx::mbar_init(&bars->empty[i], 1); }
    for (int i = 0; i < ACC_STAGES; ++i) {
      ptx::mbar_init(&bars->tmem_full[i], 1);
      ptx::mbar_init(&bars->tmem_empty[i], EPI_THREADS);
    }
    ptx::mbar_init(&bars->epi_mma, 1);
    ptx::mbar_init(&bars->epi_ops, 1);
    bars->abort = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tmap_a);
    ptx::prefetch_tmap(&tmap_b);
    if constexpr (EXT || EPI == EPI_WGRAD) { ptx::prefetch_tmap(&tmap_a2); ptx::prefetch_tmap(&tmap_b2); }
    if constexpr (TMA_STORE) ptx::prefetch_tmap(&tmap_c);
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
    // ------------------------------ TMA producer, operand A --------------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      WorkIter<TAIL_SPLIT> work(num_tiles, total_kb);
      WorkUnit u;
      while (!bars->abort && work.next(u)) {
        int tm, tn;
        tile_coords(u.tile, g.tiles_m, g.tiles_n, g.band, tm, tn);
        const int m0 = tm * BM, n0 = tn * TN;
        // (no flag check in this loop: it would be a shared-memory load on the critical path of a thread that shares
        // its scheduler with two epilogue warps; a wait that times out returns, and the abort flag ends the tile loop)
        for (int kb = u.kb0; kb < u.kb1; ++kb) {
          bounded_wait(&bars->empty[stage], phase ^ 1, bars);
          uint8_t* sa = stage_base + (size_t)stage * STAGE_BYTES;
          ptx::mbar_arrive_expect_tx(&bars->full[stage], STAGE_BYTES);   // the bytes of both operands
          // K blocks past the first operand pair come from the second one (same box shapes)
          const bool second = EXT && kb >= g.num_kb;
          const CUtensorMap* ma = second ? &tmap_a2 : &tmap_a;
          const int k0 = (second ? kb - g.num_kb : kb) * BK;
          if constexpr (!A_MN) {
            ptx::tma_load_2d(sa, ma, &bars->full[stage], k0, m0);
          } else {
#pragma unroll
            for (int h = 0; h < BM / 64; ++h)
              ptx::tma_load_2d(sa + h * (64 * BK * 2), ma, &bars->full[stage], m0 + h * 64, k0);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 2) {
    // ------------------------------ TMA producer, operand B --------------------
    // A second issuing thread: an MN-major operand takes one copy per 64 columns, and one thread issuing all of
    // a stage's copies was measurably on the critical path.  Its bytes count towards the same full barrier; they
    // may land before warp 0 has announced the stage's byte count, which the barrier's transaction count allows.
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      WorkIter<TAIL_SPLIT> work(num_tiles, total_kb);
      WorkUnit u;
      while (!bars->abort && work.next(u)) {
        int tm, tn;
        tile_coords(u.tile, g.tiles_m, g.tiles_n, g.band, tm, tn);
        const int n0 = tn * TN;
        // (no flag check in this loop: it would be a shared-memory load on the critical path of a thread that shares
        // its scheduler with two epilogue warps; a wait that times out returns, and the abort flag ends the tile loop)
        for (int kb = u.kb0; kb < u.kb1; ++kb) {
          bounded_wait(&bars->empty[stage], phase ^ 1, bars);
          uint8_t* sb = stage_base + (size_t)stage * STAGE_BYTES + A_STAGE_BYTES;
          const bool second = EXT && kb >= g.num_kb;
          const CUtensorMap* mb = second ? &tmap_b2 : &tmap_b;
          const int k0 = (second ? kb - g.num_kb : kb) * BK;
          if constexpr (!B_MN) {
            ptx::tma_load_2d(sb, mb, &bars->full[stage], k0, n0);
          } else {
#pragma unroll
            for (int h = 0; h < TN / 64; ++h)
              ptx::tma_load_2d(sb + h * (64 * BK * 2), mb, &bars->full[stage], n0 + h * 64, k0);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(BM, TN, A_MN, B_MN);
      // K-major: 8-row groups of 128-byte rows are 1024 B apart; a K step of 16 elements is +32 B.
      // MN-major: 8 k-rows of 128 bytes (64 elements along M/N) are 1024 B apart, 64-element
      // blocks along M/N are one TMA box (BK rows x 128 B) apart; a K step of 16 is two row groups.
      constexpr uint32_t A_LBO = A_MN ? (BK * 128) : 16, A_SBO = 1024, A_KSTEP = A_MN ? 2048 : 32;
      constexpr uint32_t B_LBO = B_MN ? (BK * 128) : 16, B_SBO = 1024, B_KSTEP = B_MN ? 2048 : 32;
      // This thread shares its scheduler with two epilogue warps, so every instruction here waits its turn: the
      // loop is kept to a barrier poll, one add per descriptor and the MMAs.  A descriptor's low word is the start
      // address (in 16-byte units, below 2^14) plus the leading-dimension offset, the high word is constant;
      // stages and K steps are plain increments of the low word.
      constexpr uint32_t DESC_HI = ((1024u >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);   // SBO, version 1, 128-byte swizzle
      const uint32_t a_lo0 = ((ptx::smem_u32(stage_base) >> 4) & 0x3FFFu) | (((A_LBO >> 4) & 0x3FFFu) << 16);
      const uint32_t b_lo0 = (((ptx::smem_u32(stage_base) + A_STAGE_BYTES) >> 4) & 0x3FFFu) | (((B_LBO >> 4) & 0x3FFFu) << 16);
      static_assert(A_SBO == 1024 && B_SBO == 1024, "descriptor high word");
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      WorkIter<TAIL_SPLIT> work(num_tiles, total_kb);
      WorkUnit u;
      while (!bars->abort && work.next(u)) {
        bounded_wait(&bars->tmem_empty[acc], acc_phase ^ 1, bars);
        if (bars->abort) break;
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * TN);
        uint32_t accumulate = 0;
        for (int kb = u.kb0; kb < u.kb1; ++kb) {
          bounded_wait(&bars->full[stage], phase, bars);   // on a time-out the wait returns and the abort flag ends the tile loop
          ptx::tc_fence_after_sync();
          const uint32_t al = a_lo0 + (uint32_t)stage * (STAGE_BYTES >> 4), bl = b_lo0 + (uint32_t)stage * (STAGE_BYTES >> 4);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t da = ((uint64_t)DESC_HI << 32) | (al + k * (A_KSTEP >> 4));
            const uint64_t db = ((uint64_t)DESC_HI << 32) | (bl + k * (B_KSTEP >> 4));
            ptx::mma_bf16_ss(d_tmem, da, db, idesc, accumulate);
            accumulate = 1;
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
    [[maybe_unused]] uint32_t epi_phase = 0, ops_phase = 0;
    WorkIter<TAIL_SPLIT> work(num_tiles, total_kb);
    WorkUnit u;
    while (work.next(u)) {
      int tm, tn;
      tile_coords(u.tile, g.tiles_m, g.tiles_n, g.band, tm, tn);
      const int m0 = tm * BM, n0 = tn * TN;
      const uint32_t tmem_acc = tmem_base + (uint32_t)(acc * TN);
      if constexpr (EPI == EPI_ADD_F32) {
        bounded_wait(&bars->tmem_full[acc], acc_phase, bars);
        ptx::tc_fence_after_sync();
        const int row = m0 + quarter * 32 + lane;
        constexpr int CHUNKS_PER_GROUP = (TN / 32) / EPI_GROUPS;
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
            float* dst = g.C32 + (size_t)row * g.ldc + n0 + c * 32;
#pragma unroll
            for (int e = 0; e < 32; ++e)
              if (n0 + c * 32 + e < g.N) atomicAdd(dst + e, g.scale * __uint_as_float(raw[e]));
          }
        }
      } else if constexpr (EPI == EPI_STORE && TMA_STORE) {
        bounded_wait(&bars->tmem_full[acc], acc_phase, bars);
        ptx::tc_fence_after_sync();
        const int t = quarter * 32 + lane;                       // row in tile = TMEM lane = thread of the group
        uint8_t* stg = epi_smem + eg * STORE_BOX_BYTES;
#pragma unroll 1
        for (int b = 0; b < 2; ++b) {                            // the group's 128 columns as two boxes of 64
          uint32_t raw[2][32];
          ptx::tmem_ld_32x32(tmem_acc + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(eg * 128 + b * 64), raw[0]);
          ptx::tmem_ld_32x32(tmem_acc + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(eg * 128 + b * 64 + 32), raw[1]);
          ptx::tmem_ld_wait();
          if (b == 1) {
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&bars->tmem_empty[acc]);
          }
          if (t == 0) ptx::bulk_wait_group_read0();              // the previous store has read the staging box
          ptx::named_bar_sync(1 + eg, 128);
#pragma unroll
          for (int j = 0; j < 8; ++j) {                          // 16-byte pieces of the row, 128-byte swizzle
            const uint32_t* r = raw[j >> 2] + (j & 3) * 8;
            uint4 o4;
            o4.x = pack_bf16x2(__uint_as_float(r[0]), __uint_as_float(r[1]));
            o4.y = pack_bf16x2(__uint_as_float(r[2]), __uint_as_float(r[3]));
            o4.z = pack_bf16x2(__uint_as_float(r[4]), __uint_as_float(r[5]));
            o4.w = pack_bf16x2(__uint_as_float(r[6]), __uint_as_float(r[7]));
            *reinterpret_cast<uint4*>(stg + t * 128 + ((j ^ (t & 7)) << 4)) = o4;
          }
          ptx::fence_proxy_async_smem();
          ptx::named_bar_sync(1 + eg, 128);
          // rows and columns beyond C are clipped by the copy; a box that lies outside altogether is not issued
          if (t == 0 && !bars->abort && n0 + eg * 128 + b * 64 < g.N && m0 < g.M) {
            ptx::tma_store_2d(&tmap_c, stg, n0 + eg * 128 + b * 64, m0);
            ptx::bulk_commit_group();
          }
        }
      } else if constexpr (EPI == EPI_STORE) {
        bounded_wait(&bars->tmem_full[acc], acc_phase, bars);
        ptx::tc_fence_after_sync();
        const int row = m0 + quarter * 32 + lane;
        constexpr int CHUNKS_PER_GROUP = (TN / 32) / EPI_GROUPS;
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
        if constexpr (wgrad_quarters(RANK))
          wgrad_epilogue_tile_q<RANK>(g, m0, n0, tmem_acc, quarter, lane, eg, epi_smem, bars, &bars->tmem_full[acc],
                                      acc_phase, &bars->tmem_empty[acc], epi_phase, &tmap_a2, &tmap_b2, ops_phase);
        else
          wgrad_epilogue_tile<RANK>(g, m0, n0, tmem_acc, quarter, lane, eg, epi_smem, bars, &bars->tmem_full[acc],
                                    acc_phase, &bars->tmem_empty[acc], epi_phase, &tmap_a2, &tmap_b2, ops_phase);
      }
      if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1; }
    }
  }

  // ------------------------------ teardown ------------------------------------
  if constexpr (TMA_STORE) {
    if (warp >= EPI_FIRST_WARP && (warp & 3) == 0 && lane == 0) ptx::bulk_wait_group0();   // this thread's stores have landed
  }
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

// The driver's tensor-map encoder: one entry point for the whole process, looked up once (the initialisation of a
// function-local static is thread-safe).
inline PFN_encodeTiled get_encode_fn() {
  static const PFN_encodeTiled fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<PFN_encodeTiled>(p);
  }();
  return fn;
}

// SM count and L2 size of the CURRENT device, cached per device ordinal.  Concurrent first calls may both query
// the runtime; they store the same values, and every slot is an atomic, so no caller reads a torn or foreign entry.
struct DeviceFacts {
  int sms;
  size_t l2;
};
inline DeviceFacts device_facts() {
  constexpr int kMaxDevices = 64;
  static std::atomic<int> sms[kMaxDevices];        // zero-initialised: 0 = not queried yet
  static std::atomic<size_t> l2[kMaxDevices];
  int dev = 0;
  cudaGetDevice(&dev);
  const bool cached = dev >= 0 && dev < kMaxDevices;
  DeviceFacts f{cached ? sms[dev].load(std::memory_order_acquire) : 0, cached ? l2[dev].load(std::memory_order_acquire) : 0};
  if (f.sms > 0 && f.l2 > 0) return f;
  int n = 0, bytes = 0;
  cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  cudaDeviceGetAttribute(&bytes, cudaDevAttrL2CacheSize, dev);
  f.sms = n > 0 ? n : 148;
  f.l2 = bytes > 0 ? (size_t)bytes : (size_t)96 << 20;
  if (cached) {
    l2[dev].store(f.l2, std::memory_order_release);
    sms[dev].store(f.sms, std::memory_order_release);
  }
  return f;
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

// Tile rows per band: as many A panels (128 rows x K, bf16) as fit in half of L2, the rest being left to the
// streamed operand and the output; at least 8, and split evenly so that the last band is not a sliver.
inline int tile_band_rows(int tiles_m, size_t a_panel_bytes) {
  const size_t l2 = device_facts().l2;
  int rows = (int)std::max<size_t>(8, (l2 / 2) / std::max<size_t>(a_panel_bytes, 1));
  rows = std::min(rows, tiles_m);
  const int bands = ceil_div(tiles_m, rows);
  return ceil_div(tiles_m, bands);
}

inline int sm_count() { return device_facts().sms; }

// `ta2`, `tb2`: second operand pair of an EXT launch (g.num_kb2 K blocks), or, for the weight-gradient epilogue, the
// maps of the bf16 copies of A [rn, d_in] and B^T [rn, d_out] (boxes of 64 columns x rn rows); ignored otherwise.
template <bool A_MN, bool B_MN, int EPI, int RANK, int STAGES, int TN = BN, bool EXT = false>
l4q_status launch_gemm(const CUtensorMap& ta, const CUtensorMap& tb, GemmArgs& g, cudaStream_t st,
                       const CUtensorMap* ta2 = nullptr, const CUtensorMap* tb2 = nullptr) {
  constexpr bool TMA_STORE = (EPI == EPI_STORE && TN == BN);
  CUtensorMap tc = ta;                                  // placeholder where the epilogue does not store by TMA
  if (TMA_STORE && !make_tmap_bf16(&tc, g.C, (uint64_t)g.M, (uint64_t)g.N, 128)) return cuda_fail();
  g.tiles_m = ceil_div(g.M, BM);
  g.tiles_n = ceil_div(g.N, TN);
  g.num_kb = ceil_div(g.K, BK);
  // measured: the taller band helps the GEMMs that write a large output; the weight-gradient GEMM, whose last
  // wave is cut along K, is better off with 16 rows
  g.band = EPI == EPI_STORE ? tile_band_rows(g.tiles_m, (size_t)BM * g.K * 2) : std::min(16, g.tiles_m);
  if (!EXT) g.num_kb2 = 0;
  constexpr bool SECOND_MAPS = EXT || EPI == EPI_WGRAD;   // EXT: a second operand pair; WGRAD: the bf16 copies of A and B^T
  if (SECOND_MAPS && (!ta2 || !tb2)) return L4Q_ERR_INVALID_ARG;
  auto kern = k_gemm_bf16<A_MN, B_MN, EPI, RANK, STAGES, TN, EXT>;
  const size_t smem = gemm_smem_bytes(STAGES, EPI == EPI_WGRAD ? wgrad_epi_smem_bytes(RANK)
                                              : TMA_STORE ? store_epi_smem_bytes() : 0, stage_bytes_for(TN));
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return cuda_fail();
  const int tiles = g.tiles_m * g.tiles_n, sms = sm_count();
  int grid = std::min(tiles, sms);
  if (EPI != EPI_STORE && tiles < sms) grid = tiles * std::min(sms / tiles, g.num_kb);   // K slices for the idle SMs
  kern<<<grid, GEMM_THREADS, smem, st>>>(ta, tb, SECOND_MAPS ? *ta2 : ta, SECOND_MAPS ? *tb2 : tb, tc, g);
  return cudaGetLastError() == cudaSuccess ? L4Q_OK : L4Q_ERR_CUDA;
}

// Y[tokens, d_out] = X[tokens, d_in] Wq[d_out, d_in]^T
inline l4q_status gemm_forward_bf16(const Params& p, const void* X, const void* Wq, void* Y, cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!make_tmap_bf16(&ta, X, p.tokens, p.d_in, BM) || !make_tmap_bf16(&tb, Wq, p.d_out, p.d_in, BN))
    return cuda_fail();
  GemmArgs g{};
  g.M = p.tokens; g.N = p.d_out; g.K = p.d_in;
  g.C = reinterpret_cast<__nv_bfloat16*>(Y);
  return launch_gemm<false, false, EPI_STORE, 0, 4>(ta, tb, g, st);
}

// dX[tokens, d_in] = dY[tokens, d_out] Wq[d_out, d_in]
inline l4q_status gemm_dgrad_bf16(const Params& p, const void* dY, const void* Wq, void* dX, cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!make_tmap_bf16(&ta, dY, p.tokens, p.d_out, BM) || !make_tmap_bf16(&tb, Wq, p.d_out, p.d_in, BK))
    return cuda_fail();
  GemmArgs g{};
  g.M = p.tokens; g.N = p.d_in; g.K = p.d_out;
  g.C = reinterpret_cast<__nv_bfloat16*>(dX);
  return launch_gemm<false, true, EPI_STORE, 0, 4>(ta, tb, g, st);
}

// G[d_out, d_in] = dY^T X reduced on chip into dA, dB, ds, db (which must be zero on entry).
// A16 [rn, d_in], Bt16 [rn, d_out]: bf16 copies of A and B^T with rn = wgrad_rn(rank) rows, rows beyond the rank zero.
inline l4q_status gemm_wgrad_bf16(const Params& p, const void* X, const void* dY, const void* F, const void* A16,
                                  const void* Bt16, float* dA, float* dB, float* ds, float* db, cudaStream_t st) {
  CUtensorMap ta, tb, ta16, tbt16;
  const int rn = wgrad_rn(p.rank);
  if (!make_tmap_bf16(&ta, dY, p.tokens, p.d_out, BK) || !make_tmap_bf16(&tb, X, p.tokens, p.d_in, BK) ||
      !make_tmap_bf16(&ta16, A16, rn, p.d_in, rn) || !make_tmap_bf16(&tbt16, Bt16, rn, p.d_out, rn))
    return cuda_fail();
  GemmArgs g{};
  g.M = p.d_out; g.N = p.d_in; g.K = p.tokens;
  g.p = p;
  g.F = reinterpret_cast<const __half*>(F);
  g.f_tiles_n = factor_tiles_n(p.d_in);
  g.dA = dA; g.dB = dB; g.ds = ds; g.db = db;
  switch (p.rank) {
    case 8: return launch_gemm<true, true, EPI_WGRAD, 8, wgrad_stages(8)>(ta, tb, g, st, &ta16, &tbt16);
    case 16: return launch_gemm<true, true, EPI_WGRAD, 16, wgrad_stages(16)>(ta, tb, g, st, &ta16, &tbt16);
    case 32: return launch_gemm<true, true, EPI_WGRAD, 32, 3>(ta, tb, g, st, &ta16, &tbt16);
    case 64: return launch_gemm<true, true, EPI_WGRAD, 64, 3>(ta, tb, g, st, &ta16, &tbt16);
    default: return L4Q_ERR_UNSUPPORTED;
  }
}

}  // namespace l4q
