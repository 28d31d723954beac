// Weight-tile kernel of the bf16 path: merge (Eq. 7) + fake-quantize (Eq. 8-9) the weight in
// 128 x 128 tiles, streaming W0 once from HBM, and write one of
//   WT2_DEQUANT    W_q (bf16)                      -- the recompute step of forward and backward (App. E.2)
//   WT2_DEQUANT_F  W_q (bf16) + STE factors (fp16) -- backward: input gradient + weight-gradient reduction
//   WT2_PACK       bit-packed codes + fp16 s, b    -- export (Sec. 3.2)
//
// HBM-bound by design (2 bytes in, 2-4 bytes out per weight), so everything else is arranged to stay out
// of the way of the copies:
//   * W0 tiles arrive by TMA into 128-byte-swizzled shared memory (2-4 stages in flight); W_q is written
//     back IN PLACE into the same stage and leaves by a TMA store, so every global access is a full line;
//   * the rank-r merge B A is a tensor-core contraction: tcgen05.mma kind::tf32 into tensor memory, with
//     each fp32 factor split into a tf32 head and a tf32 tail (x = hi + lo, three products hi*hi + hi*lo +
//     lo*hi), which keeps ~21 mantissa bits -- the codes must agree with fp64 arithmetic except within
//     1e-6 of a rounding boundary, which a single tf32 or bf16 product does not give;
//   * 16 epilogue warps (thread = one weight row x 32 columns) read the merge from tensor memory with
//     tcgen05.ld, the W0 tile from shared memory in 16-byte pieces, and do the quantizer arithmetic.
//
// Roles (640 threads): warp 0 = TMA loads, warp 1 = MMA issuer + TMEM owner, warp 2 = TMA stores,
// warps 4..19 = epilogue (warp w: TMEM lane quarter w % 4, column slice (w - 4) / 4).  The epilogue warps
// also build the split LoRA operands of the NEXT tile as soon as the MMAs of the current one have
// completed, so the merge of tile t + 1 overlaps the quantizer arithmetic of tile t.
// Every wait is bounded (see bounded_wait).
#pragma once

#include "l4q_common.cuh"
#include "l4q_gemm.cuh"
#include "l4q_ptx.cuh"

namespace l4q {

constexpr int WT2_ROWS = 128, WT2_COLS = 128;
constexpr int WT2_THREADS = 640;
constexpr int WT2_FIRST_EPI_WARP = 4;
constexpr int WT2_EPI_THREADS = 512;
constexpr int WT2_ACC = 4;                          // accumulator stages of 128 TMEM columns
constexpr int WT2_STAGE_BYTES = WT2_ROWS * WT2_COLS * 2;   // one bf16 tile: two 128 x 64 swizzled boxes
constexpr int WT2_ATOM_BYTES = 128 * 128;           // 128 rows x 32 tf32 (one 128-byte swizzle atom along K)
constexpr int WT2_MAX_STAGES = 4;

enum { WT2_DEQUANT = 0, WT2_DEQUANT_F = 1, WT2_PACK = 2 };

struct WtileArgs {
  Params p;
  const float *A, *B, *s, *b;
  __half *s16, *b16;       // WT2_PACK
  int tiles_m, tiles_n;
  int n_stages;            // W0 stages in shared memory (2..4)
  int n_out;               // staging buffers for the second output (F or codes): 0, 1 or 2
  int out_bytes;           // bytes of one such buffer
  int atoms;               // swizzle atoms per operand row: ceil(2 rank / 32)
  int ngt;                 // upper bound of the quantization groups a 128-column tile intersects
};

struct __align__(8) WtileBarriers {
  uint64_t full[WT2_MAX_STAGES];      // W0 tile has landed in the stage
  uint64_t empty[WT2_MAX_STAGES];     // the stage may be overwritten (its store has read it)
  uint64_t written[WT2_MAX_STAGES];   // the epilogue has written the stage's outputs
  uint64_t out_empty[2];              // second-output staging buffer may be overwritten
  uint64_t prep_full;                 // split LoRA operands of the next tile are in shared memory
  uint64_t tmem_full[WT2_ACC], tmem_empty[WT2_ACC];
  uint32_t tmem_base;
  volatile uint32_t abort;
};

// s and b of a tile in shared memory: two buffers of [128 rows][s x ngt | b x ngt] floats (1 KB multiples).
__host__ __device__ inline size_t wtile_sb_bytes(int ngt) { return 2 * (size_t)WT2_ROWS * 2 * ngt * sizeof(float); }

inline size_t wtile_smem_bytes(const WtileArgs& a) {
  return 1024 + (size_t)a.n_stages * WT2_STAGE_BYTES + (size_t)a.n_out * a.out_bytes +
         2 * (size_t)a.atoms * WT2_ATOM_BYTES + wtile_sb_bytes(a.ngt) + sizeof(WtileBarriers);
}

// Tile i of this CTA: row tiles of one column panel go to neighbouring CTAs.
__device__ __forceinline__ bool wtile_coords(const WtileArgs& a, int i, int& m0, int& n0) {
  const int t = blockIdx.x + i * gridDim.x;
  if (t >= a.tiles_m * a.tiles_n) return false;
  m0 = (t % a.tiles_m) * WT2_ROWS;
  n0 = (t / a.tiles_m) * WT2_COLS;
  return true;
}

// x = hi + lo with hi, lo representable in tf32 (low 13 mantissa bits clear): hi keeps the leading 10
// mantissa bits of x (truncation), lo the leading bits of the exact remainder.  Plain logic ops.
__device__ __forceinline__ void split_tf32(float x, float& hi, float& lo) {
  hi = __uint_as_float(__float_as_uint(x) & 0xFFFFE000u);
  lo = __uint_as_float(__float_as_uint(x - hi) & 0xFFFFE000u);
}

// Builds the split operands of one tile in shared memory, K-major with the 128-byte swizzle:
//   acat row n = column n0 + n of the weight:  [ hi(A[0..r, col]) | lo(A[0..r, col]) ]
//   bcat row m = row m0 + m of the weight:      [ hi(B[row, 0..r]) | lo(B[row, 0..r]) ]
// A work item is 4 consecutive ranks of one row; a warp takes 32 consecutive rows of the same ranks, so
// its reads of A are coalesced and its 16-byte shared-memory writes are conflict-free.
__device__ __forceinline__ void wtile_prep_operands(const WtileArgs& a, int m0, int n0, int et, uint8_t* acat,
                                                    uint8_t* bcat) {
  const Params& p = a.p;
  const int r = p.rank;
  for (int idx = et; idx < 32 * r; idx += WT2_EPI_THREADS) {
    const int row = idx & 127, kc = idx >> 7;        // ranks 4 kc .. 4 kc + 3
    float av[4] = {0.f, 0.f, 0.f, 0.f};
    const int col = n0 + row;
    if (col < p.d_in) {
#pragma unroll
      for (int e = 0; e < 4; ++e) av[e] = __ldg(a.A + (size_t)(4 * kc + e) * p.d_in + col);
    }
    float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
    if (m0 + row < p.d_out) bv = __ldg(reinterpret_cast<const float4*>(a.B + (size_t)(m0 + row) * r + 4 * kc));
    const float bvv[4] = {bv.x, bv.y, bv.z, bv.w};
    float ah[4], al[4], bh[4], bl[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      split_tf32(av[e], ah[e], al[e]);
      split_tf32(bvv[e], bh[e], bl[e]);
    }
    const int ch = kc, cl = (r >> 2) + kc;           // 16-byte chunk index of the head / tail within the row
    const uint32_t off_h = (uint32_t)(ch >> 3) * WT2_ATOM_BYTES + row * 128 + (((ch & 7) ^ (row & 7)) << 4);
    const uint32_t off_l = (uint32_t)(cl >> 3) * WT2_ATOM_BYTES + row * 128 + (((cl & 7) ^ (row & 7)) << 4);
    *reinterpret_cast<float4*>(acat + off_h) = make_float4(ah[0], ah[1], ah[2], ah[3]);
    *reinterpret_cast<float4*>(acat + off_l) = make_float4(al[0], al[1], al[2], al[3]);
    *reinterpret_cast<float4*>(bcat + off_h) = make_float4(bh[0], bh[1], bh[2], bh[3]);
    *reinterpret_cast<float4*>(bcat + off_l) = make_float4(bl[0], bl[1], bl[2], bl[3]);
  }
}

// 32 unsigned codes -> bitstream words, code j at bit j * BITS (LSB first).
template <int BITS>
__device__ __forceinline__ void pack_codes32(const uint32_t (&u)[32], uint32_t (&w)[BITS]) {
#pragma unroll
  for (int i = 0; i < BITS; ++i) w[i] = 0u;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const int bit = j * BITS, word = bit >> 5, off = bit & 31;
    w[word] |= u[j] << off;
    if (off + BITS > 32) w[word + 1] |= u[j] >> (32 - off);
  }
}

template <int MODE>
__global__ void __launch_bounds__(WT2_THREADS, 1)
k_wtile_tc(const __grid_constant__ CUtensorMap tmap_w0,     // load:  W0 [d_out, d_in] bf16, box 64 x 128, swizzled
           const __grid_constant__ CUtensorMap tmap_out0,   // store: W_q (same geometry) | codes (uint32 words)
           const __grid_constant__ CUtensorMap tmap_out1,   // store: STE factors (same geometry as W0) | unused
           const WtileArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* stage_base = smem;
  uint8_t* out_base = stage_base + (size_t)a.n_stages * WT2_STAGE_BYTES;
  uint8_t* acat = out_base + (size_t)a.n_out * a.out_bytes;
  uint8_t* bcat = acat + (size_t)a.atoms * WT2_ATOM_BYTES;
  float* sb_base = reinterpret_cast<float*>(bcat + (size_t)a.atoms * WT2_ATOM_BYTES);
  WtileBarriers* bars = reinterpret_cast<WtileBarriers*>(reinterpret_cast<uint8_t*>(sb_base) + wtile_sb_bytes(a.ngt));
  const Params& p = a.p;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr bool HAS_OUT1 = (MODE != WT2_DEQUANT);

  if (threadIdx.x == 0) {
    for (int i = 0; i < WT2_MAX_STAGES; ++i) {
      ptx::mbar_init(&bars->full[i], 1);
      ptx::mbar_init(&bars->empty[i], 1);
      ptx::mbar_init(&bars->written[i], WT2_EPI_THREADS);
    }
    for (int i = 0; i < 2; ++i) ptx::mbar_init(&bars->out_empty[i], 1);
    ptx::mbar_init(&bars->prep_full, WT2_EPI_THREADS);
    for (int i = 0; i < WT2_ACC; ++i) {
      ptx::mbar_init(&bars->tmem_full[i], 1);
      ptx::mbar_init(&bars->tmem_empty[i], WT2_EPI_THREADS);
    }
    bars->abort = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tmap_w0);
    ptx::prefetch_tmap(&tmap_out0);
    if (MODE == WT2_DEQUANT_F) ptx::prefetch_tmap(&tmap_out1);
  }
  if (warp == 1) {
    ptx::tmem_alloc(&bars->tmem_base, WT2_ACC * WT2_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;

  if (warp == 0) {
    // ------------------------------ TMA loads of W0 ---------------------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      int m0, n0;
      for (int i = 0; !bars->abort && wtile_coords(a, i, m0, n0); ++i) {
        bounded_wait(&bars->empty[stage], phase ^ 1, bars);
        if (bars->abort) break;
        uint8_t* dst = stage_base + (size_t)stage * WT2_STAGE_BYTES;
        ptx::mbar_arrive_expect_tx(&bars->full[stage], WT2_STAGE_BYTES);
        ptx::tma_load_2d(dst, &tmap_w0, &bars->full[stage], n0, m0);
        ptx::tma_load_2d(dst + WT2_STAGE_BYTES / 2, &tmap_w0, &bars->full[stage], n0 + 64, m0);
        if (++stage == a.n_stages) { stage = 0; phase ^= 1; }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------ merge MMAs --------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_tf32(WT2_ROWS, WT2_COLS);
      const uint32_t acat_a = ptx::smem_u32(acat), bcat_a = ptx::smem_u32(bcat);
      const int r = p.rank, ksteps = r >> 3;
      int acc = 0; uint32_t acc_phase = 0;
      int m0, n0;
      for (int i = 0; !bars->abort && wtile_coords(a, i, m0, n0); ++i) {
        bounded_wait(&bars->prep_full, (uint32_t)(i & 1), bars);
        bounded_wait(&bars->tmem_empty[acc], acc_phase ^ 1, bars);
        if (bars->abort) break;
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * WT2_COLS);
        uint32_t accumulate = 0;
        // B A = Bhi Ahi + Bhi Alo + Blo Ahi  (the tail x tail product is below fp32 resolution of the sum)
#pragma unroll 1
        for (int term = 0; term < 3; ++term) {
          const int eb0 = (term == 2) ? r : 0;       // element offset into the B rows (M operand)
          const int ea0 = (term == 1) ? r : 0;       // element offset into the A rows (N operand)
          for (int ks = 0; ks < ksteps; ++ks) {
            const int eb = eb0 + ks * 8, ea = ea0 + ks * 8;
            const uint64_t dm = ptx::make_smem_desc_sw128(bcat_a + (eb >> 5) * WT2_ATOM_BYTES + (eb & 31) * 4, 16, 1024);
            const uint64_t dn = ptx::make_smem_desc_sw128(acat_a + (ea >> 5) * WT2_ATOM_BYTES + (ea & 31) * 4, 16, 1024);
            ptx::mma_tf32_ss(d_tmem, dm, dn, idesc, accumulate);
            accumulate = 1;
          }
        }
        ptx::mma_commit(&bars->tmem_full[acc]);
        if (++acc == WT2_ACC) { acc = 0; acc_phase ^= 1; }
      }
    }
    __syncwarp();
  } else if (warp == 2) {
    // ------------------------------ TMA stores --------------------------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      int ob = 0;
      int m0, n0;
      for (int i = 0; !bars->abort && wtile_coords(a, i, m0, n0); ++i) {
        bounded_wait(&bars->written[stage], phase, bars);
        if (bars->abort) break;
        const uint8_t* src = stage_base + (size_t)stage * WT2_STAGE_BYTES;
        const uint8_t* src1 = out_base + (size_t)ob * a.out_bytes;
        const bool second_box = n0 + 64 < p.d_in;
        if constexpr (MODE != WT2_PACK) {
          ptx::tma_store_2d(&tmap_out0, src, n0, m0);
          if (second_box) ptx::tma_store_2d(&tmap_out0, src + WT2_STAGE_BYTES / 2, n0 + 64, m0);
        }
        if constexpr (MODE == WT2_DEQUANT_F) {
          ptx::tma_store_2d(&tmap_out1, src1, n0, m0);
          if (second_box) ptx::tma_store_2d(&tmap_out1, src1 + WT2_STAGE_BYTES / 2, n0 + 64, m0);
        }
        if constexpr (MODE == WT2_PACK) ptx::tma_store_2d(&tmap_out0, src1, (n0 * p.bits) >> 5, m0);
        ptx::bulk_commit_group();
        ptx::bulk_wait_group_read0();
        ptx::mbar_arrive(&bars->empty[stage]);
        if constexpr (HAS_OUT1) {
          ptx::mbar_arrive(&bars->out_empty[ob]);
          if (++ob == a.n_out) ob = 0;
        }
        if (++stage == a.n_stages) { stage = 0; phase ^= 1; }
      }
      ptx::bulk_wait_group0();
    }
    __syncwarp();
  } else if (warp >= WT2_FIRST_EPI_WARP) {
    // ------------------------------ epilogue ----------------------------------
    const int quarter = warp & 3;
    const int sl = (warp - WT2_FIRST_EPI_WARP) >> 2;            // 32-column slice of the tile
    const int row = quarter * 32 + lane;
    const int et = (warp - WT2_FIRST_EPI_WARP) * 32 + lane;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    int stage = 0; uint32_t phase = 0;
    int acc = 0; uint32_t acc_phase = 0;
    int ob = 0; uint32_t out_round = 0;                         // uses of staging buffer `ob` so far
    int m0, n0;
    // s and b reach the arithmetic through shared memory: the four warps of column slice 0 (one thread
    // per weight row) copy the tile's values of their row, one tile ahead, with asynchronous 4-byte
    // copies; all epilogue threads meet at a barrier at the end of every tile.  (Loading them per thread
    // would touch 32 different lines per instruction, sixteen times over, and starve the TMA loads.)
    const int sbw = 2 * a.ngt;                                  // floats per row: s x ngt | b x ngt
    auto stage_sb = [&](int m0_, int n0_, int buf) {
      if (sl != 0) return;
      float* dst = sb_base + ((size_t)buf * WT2_ROWS + row) * sbw;
      const int o_ = m0_ + row;
      const int g_first = n0_ / p.group;
      for (int k = 0; k < a.ngt; ++k) {
        const int g = g_first + k;
        if (o_ < p.d_out && g < p.ngroups) {
          ptx::cp_async_4(dst + k, a.s + (size_t)o_ * p.ngroups + g);
          ptx::cp_async_4(dst + a.ngt + k, a.b + (size_t)o_ * p.ngroups + g);
        } else {
          dst[k] = 1.f; dst[a.ngt + k] = 0.f;
        }
      }
      ptx::cp_async_commit();
    };
    if (wtile_coords(a, 0, m0, n0)) {
      stage_sb(m0, n0, 0);
      wtile_prep_operands(a, m0, n0, et, acat, bcat);
      ptx::fence_proxy_async_smem();
      ptx::mbar_arrive(&bars->prep_full);
      ptx::cp_async_wait_all();
    }
    ptx::named_bar_sync(1, WT2_EPI_THREADS);
    for (int i = 0; wtile_coords(a, i, m0, n0); ++i) {
      const int o = m0 + row;
      const bool row_ok = o < p.d_out;
      const int jc = n0 + sl * 32;
      float sv[4], bv[4];
      int grp[4];
      uint32_t first_mask = 0;                                  // bit sub: the piece is the first of its group
      {
        const int g_first = n0 / p.group;
        const int g0 = jc / p.group;
        const int rem0 = jc - g0 * p.group;
        const float* src = sb_base + ((size_t)(i & 1) * WT2_ROWS + row) * sbw;
#pragma unroll
        for (int sub = 0; sub < 4; ++sub) {
          int rem = rem0 + sub * 8, g = g0;
#pragma unroll
          for (int c = 0; c < 3; ++c)
            if (rem >= p.group) { rem -= p.group; ++g; }
          const bool ok = row_ok && jc + sub * 8 < p.d_in;
          grp[sub] = ok ? g : -1;
          if (rem == 0) first_mask |= 1u << sub;
          sv[sub] = ok ? src[g - g_first] : 1.f;
          bv[sub] = ok ? src[a.ngt + g - g_first] : 0.f;
        }
      }
      bounded_wait(&bars->tmem_full[acc], acc_phase, bars);
      ptx::tc_fence_after_sync();
      {  // the MMAs of this tile have completed: their operands may be replaced by the next tile's
        int m1, n1;
        if (wtile_coords(a, i + 1, m1, n1)) {
          stage_sb(m1, n1, (i + 1) & 1);
          wtile_prep_operands(a, m1, n1, et, acat, bcat);
          ptx::fence_proxy_async_smem();
          ptx::mbar_arrive(&bars->prep_full);
        }
      }
      uint32_t raw[32];
      ptx::tmem_ld_32x32(tmem_base + lane_base + (uint32_t)(acc * WT2_COLS + sl * 32), raw);
      ptx::tmem_ld_wait();
      ptx::tc_fence_before_sync();
      ptx::mbar_arrive(&bars->tmem_empty[acc]);

      bounded_wait(&bars->full[stage], phase, bars);
      if constexpr (HAS_OUT1) {
        if (out_round > 0) bounded_wait(&bars->out_empty[ob], (out_round - 1) & 1, bars);
      }
      uint8_t* wrow = stage_base + (size_t)stage * WT2_STAGE_BYTES + (sl >> 1) * (WT2_STAGE_BYTES / 2) + row * 128;
      [[maybe_unused]] uint8_t* out1 = out_base + (size_t)ob * a.out_bytes;
      [[maybe_unused]] uint32_t ucodes[32];
      float rs = 1.f;
#pragma unroll
      for (int sub = 0; sub < 4; ++sub) {
        const uint32_t chunk = (uint32_t)((((sl & 1) * 4 + sub) ^ (row & 7)) << 4);
        const uint4 wr = *reinterpret_cast<const uint4*>(wrow + chunk);
        const float w0[8] = {bf16_lo(wr.x), bf16_hi(wr.x), bf16_lo(wr.y), bf16_hi(wr.y),
                             bf16_lo(wr.z), bf16_hi(wr.z), bf16_lo(wr.w), bf16_hi(wr.w)};
        if (sub == 0 || ((first_mask >> sub) & 1u)) rs = 1.0f / sv[sub];         // one reciprocal per group
        float wq[8], fac[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const QuantElem q = quantize_elem(merge_elem(w0[e], __uint_as_float(raw[sub * 8 + e]), p.gamma), sv[sub], rs,
                                            bv[sub], p.qn, p.qp);
          wq[e] = q.wq;
          fac[e] = ste_factor(q, p.qn, p.qp);
          if constexpr (MODE == WT2_PACK) ucodes[sub * 8 + e] = (uint32_t)(int)(q.code - p.qn);
        }
        if constexpr (MODE != WT2_PACK) {
          uint4 o4;
          o4.x = pack_bf16x2(wq[0], wq[1]); o4.y = pack_bf16x2(wq[2], wq[3]);
          o4.z = pack_bf16x2(wq[4], wq[5]); o4.w = pack_bf16x2(wq[6], wq[7]);
          *reinterpret_cast<uint4*>(wrow + chunk) = o4;                       // in place, same swizzled position
        }
        if constexpr (MODE == WT2_DEQUANT_F) {
          __half2 h[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) h[e] = __floats2half2_rn(fac[2 * e], fac[2 * e + 1]);
          *reinterpret_cast<uint4*>(out1 + (sl >> 1) * (WT2_STAGE_BYTES / 2) + row * 128 + chunk) =
              *reinterpret_cast<const uint4*>(h);
        }
        if constexpr (MODE == WT2_PACK) {
          if (grp[sub] >= 0 && ((first_mask >> sub) & 1u)) {                   // first piece of its group
            a.s16[(size_t)o * p.ngroups + grp[sub]] = __float2half_rn(sv[sub]);
            a.b16[(size_t)o * p.ngroups + grp[sub]] = __float2half_rn(fmaf(sv[sub], p.qn, bv[sub]));
          }
        }
      }
      if constexpr (MODE == WT2_PACK) {
        // staging row = the tile's 128 codes of this weight row; this thread owns 32 of them
        if (p.bits == 4) {
          uint32_t w[4];
          pack_codes32<4>(ucodes, w);
          *reinterpret_cast<uint4*>(out1 + row * 64 + sl * 16) = make_uint4(w[0], w[1], w[2], w[3]);
        } else {
          uint32_t w[3];
          pack_codes32<3>(ucodes, w);
          uint32_t* dst = reinterpret_cast<uint32_t*>(out1 + row * 48 + sl * 12);
          dst[0] = w[0]; dst[1] = w[1]; dst[2] = w[2];
        }
      }
      ptx::fence_proxy_async_smem();                   // the stores above are read by TMA
      ptx::mbar_arrive(&bars->written[stage]);
      ptx::cp_async_wait_all();                        // this thread's copies of the next tile's s, b have landed
      ptx::named_bar_sync(1, WT2_EPI_THREADS);         // ... and so have everyone's
      if (++stage == a.n_stages) { stage = 0; phase ^= 1; }
      if (++acc == WT2_ACC) { acc = 0; acc_phase ^= 1; }
      if constexpr (HAS_OUT1) {
        if (++ob == a.n_out) { ob = 0; ++out_round; }
      }
    }
  }

  // ------------------------------ teardown ------------------------------------
  if (bars->abort) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);  // let copies in flight land before shared memory is released
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, WT2_ACC * WT2_COLS);
  }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------

// uint32 row-major matrix [rows, words]; box = [box_words, 128 rows], no swizzle (code words of the export).
inline bool make_tmap_words(CUtensorMap* m, const void* base, uint64_t rows, uint64_t words, uint32_t box_words) {
  PFN_encodeTiled enc = get_encode_fn();
  if (!enc) return false;
  const cuuint64_t gdim[2] = {words, rows};
  const cuuint64_t gstride[1] = {words * 4};
  const cuuint32_t box[2] = {box_words, 128};
  const cuuint32_t estr[2] = {1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(base), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Shared-memory plan: LoRA operands first, then as many W0 stages as fit (a second staging buffer for
// the extra output only if three stages still fit beside it).
inline bool wtile_plan(WtileArgs& a, int mode) {
  const Params& p = a.p;
  a.atoms = (2 * p.rank + 31) / 32;
  a.ngt = std::min(p.ngroups, (WT2_COLS - 1) / p.group + 2);
  a.out_bytes = mode == WT2_DEQUANT_F ? WT2_STAGE_BYTES : mode == WT2_PACK ? WT2_ROWS * (WT2_COLS * p.bits / 8) : 0;
  const long long budget = 227 * 1024 - 1024 - (long long)sizeof(WtileBarriers) - 2LL * a.atoms * WT2_ATOM_BYTES -
                           (long long)wtile_sb_bytes(a.ngt);
  a.n_out = a.out_bytes ? 2 : 0;
  long long stages = (budget - (long long)a.n_out * a.out_bytes) / WT2_STAGE_BYTES;
  if (a.n_out == 2 && stages < 3) {
    a.n_out = 1;
    stages = (budget - a.out_bytes) / WT2_STAGE_BYTES;
  }
  if (stages < 2) return false;
  a.n_stages = (int)std::min<long long>(stages, WT2_MAX_STAGES);
  return true;
}

// Whether the tensor-core weight-tile kernel covers this problem (otherwise the plain-ALU kernel runs).
inline bool wtile_tc_supported(const Params& p, int mode) {
  if (p.rank % 8 != 0 || p.rank > 64) return false;
  if (mode == WT2_PACK) {
    if (p.bits != 3 && p.bits != 4) return false;
    const long long words = ((long long)p.d_in * p.bits) >> 5;
    if (((long long)p.d_in * p.bits) % 32 != 0 || (words * 4) % 16 != 0) return false;   // TMA row pitch
  }
  WtileArgs a{};
  a.p = p;
  return wtile_plan(a, mode);                       // the shared-memory plan must fit (rank 64 with the factor output does not)
}

// mode WT2_DEQUANT: out0 = W_q.  WT2_DEQUANT_F: out0 = W_q, out1 = STE factors.  WT2_PACK: out0 = codes.
inline l4q_status launch_wtile_tc(int mode, const Params& p, const void* W0, const float* A, const float* B,
                                  const float* s, const float* b, void* out0, void* out1, __half* s16, __half* b16,
                                  cudaStream_t st) {
  WtileArgs a{};
  a.p = p; a.A = A; a.B = B; a.s = s; a.b = b; a.s16 = s16; a.b16 = b16;
  a.tiles_m = ceil_div(p.d_out, WT2_ROWS);
  a.tiles_n = ceil_div(p.d_in, WT2_COLS);
  if (!wtile_plan(a, mode)) return L4Q_ERR_UNSUPPORTED;
  CUtensorMap t_w0, t_o0, t_o1;
  if (!make_tmap_bf16(&t_w0, W0, p.d_out, p.d_in, WT2_ROWS)) return L4Q_ERR_CUDA;
  t_o1 = t_w0;
  if (mode == WT2_PACK) {
    if (!make_tmap_words(&t_o0, out0, p.d_out, ((uint64_t)p.d_in * p.bits) >> 5, WT2_COLS * p.bits / 32))
      return L4Q_ERR_CUDA;
  } else {
    if (!make_tmap_bf16(&t_o0, out0, p.d_out, p.d_in, WT2_ROWS)) return L4Q_ERR_CUDA;
    if (mode == WT2_DEQUANT_F && !make_tmap_bf16(&t_o1, out1, p.d_out, p.d_in, WT2_ROWS)) return L4Q_ERR_CUDA;
  }
  const size_t smem = wtile_smem_bytes(a);
  const int grid = std::min(a.tiles_m * a.tiles_n, sm_count());
  auto launch = [&](auto kern) -> l4q_status {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return L4Q_ERR_CUDA;
    kern<<<grid, WT2_THREADS, smem, st>>>(t_w0, t_o0, t_o1, a);
    return cudaGetLastError() == cudaSuccess ? L4Q_OK : L4Q_ERR_CUDA;
  };
  switch (mode) {
    case WT2_DEQUANT: return launch(k_wtile_tc<WT2_DEQUANT>);
    case WT2_DEQUANT_F: return launch(k_wtile_tc<WT2_DEQUANT_F>);
    default: return launch(k_wtile_tc<WT2_PACK>);
  }
}

}  // namespace l4q
