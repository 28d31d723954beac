// Fully quantized inference (Sec. 3.2, App. F): Y = X W_q^T where only the export of l4q_pack_int is
// kept -- bit-packed unsigned codes u and one fp16 scale / offset per group, W_q = u * s16 + b16.
//
// The regime of the paper's deployment measurements is a handful of tokens per step (batch 1..64), so the
// kernel is bound by reading the packed weight once (bits/8 bytes per weight) and is built around that:
//   * tokens are the MMA's M (one 128-row tile, zero-filled beyond the batch), output features its N, in
//     tiles of 64 rows of W so that even a 4096-row layer gives every SM work;
//   * the packed code words of a tile (N rows x 64 or 48 bytes per 128-deep k-step) arrive by TMA through a
//     deep ring (8 steps in flight: they are the only HBM traffic), the X tile (128-byte-swizzled, from L2)
//     and the dequantized operand through a shallow one (3 steps);
//   * up to 384 dequantizer threads (one per weight row and 32 codes) turn the words into bf16 W_q = u * s + b
//     (fp32 arithmetic) and write the MMA's B operand in the swizzled K-major layout; one thread issues
//     tcgen05.mma (bf16 x bf16 -> fp32 in tensor memory);
//   * 4 epilogue warps drain the 128 x N accumulator of the previous tile meanwhile;
//   * N (16..96 weight rows per tile) is chosen per layer so that the tiles fill whole waves of SMs.
// Roles (640 threads): warp 0 = TMA of X, warp 2 = TMA of the code words, warp 1 = MMA issuer + TMEM owner,
// warps 4..7 = epilogue, warps 8..19 = dequantizers.  Every mbarrier wait is bounded (bounded_wait).
#pragma once

#include "l4q_common.cuh"
#include "l4q_gemm.cuh"
#include "l4q_ptx.cuh"
#include "l4q_wtile.cuh"

namespace l4q {

constexpr int INF_M = 128;                 // tokens per tile (MMA M)
constexpr int INF_NMAX = 96;               // most weight rows per tile (MMA N, a multiple of 16 chosen per problem)
constexpr int INF_BK = 128;                // k per pipeline step
constexpr int INF_OP_STAGES = 3;           // X tile + dequantized W tile
constexpr int INF_C_STAGES = 8;            // packed code words, loaded far ahead: they are what comes from HBM
constexpr int INF_THREADS = 640;
constexpr int INF_DEQ_THREADS = 384;       // warps 8..19: one thread per (weight row, 32 codes) unit, 4 * INF_NMAX
constexpr int INF_X_BYTES = INF_M * INF_BK * 2;         // 32 KB: two 128 x 64 swizzled boxes
constexpr int INF_W_BYTES = INF_NMAX * INF_BK * 2;      // 24 KB reserved: two (N x 64) swizzled tiles, 12 KB apart
constexpr int INF_OP_BYTES = INF_X_BYTES + INF_W_BYTES;
constexpr int INF_C_BYTES = INF_NMAX * 16 * 4;          // 6 KB reserved: N rows x (16 | 12) words
constexpr int INF_ACC = 2;
constexpr int INF_ACC_COLS = 128;          // TMEM columns per accumulator stage

struct InferArgs {
  int tokens, d_in, d_out, bits, group, ngroups;
  int tile_n;                              // weight rows per tile
  int group_shift;                         // log2(group size) if it is a power of two, else -1
  int x_rows;                              // token rows a TMA box of X brings in (8 .. 128)
  int tiles_m, tiles_n, num_kb;
  const __half *s16, *b16;
  __nv_bfloat16* Y;
};

struct __align__(8) InferBarriers {
  uint64_t full_x[INF_OP_STAGES];          // X tile has landed
  uint64_t full_w[INF_OP_STAGES];          // the dequantized B operand of the stage is complete
  uint64_t empty_op[INF_OP_STAGES];        // the MMAs reading the operand stage have completed
  uint64_t full_c[INF_C_STAGES];           // code words have landed
  uint64_t empty_c[INF_C_STAGES];          // the dequantizers have read the code words
  uint64_t tmem_full[INF_ACC], tmem_empty[INF_ACC];
  uint32_t tmem_base;
  volatile uint32_t abort;
};

inline size_t infer_smem_bytes() {
  return 1024 + (size_t)INF_OP_STAGES * INF_OP_BYTES + (size_t)INF_C_STAGES * INF_C_BYTES + sizeof(InferBarriers);
}

// 32 unsigned codes of one weight row (starting at a multiple of 32 codes of the LSB-first bitstream), each
// returned as the float m = 1 + u / 2^BITS: the code is moved into the top mantissa bits under the exponent
// of 1.0 (one shift and one logic op, no integer-to-float conversion).  The caller folds the affine map back:
// u * s + b = m * (2^BITS s) + (b - 2^BITS s), a single fma.
template <int BITS>
__device__ __forceinline__ float unpack_code(const uint32_t (&w)[BITS], int j) {      // j: compile-time after unrolling
  constexpr int POS = 23 - BITS;                               // bit position of the code inside the mantissa
  constexpr uint32_t MASK = ((1u << BITS) - 1u) << POS;
  const int bit = j * BITS, wd = bit >> 5, off = bit & 31;
  uint32_t v;
  if (off + BITS > 32) v = __funnelshift_r(w[wd], w[wd + 1 < BITS ? wd + 1 : wd], off) << POS;   // code straddles two words
  else v = (off <= POS) ? (w[wd] << (POS - off)) : (w[wd] >> (off - POS));
  return __uint_as_float((v & MASK) | 0x3F800000u);
}

template <int BITS>
__device__ __forceinline__ void unpack_codes32(const uint32_t (&w)[BITS], float (&m)[32]) {
#pragma unroll
  for (int j = 0; j < 32; ++j) m[j] = unpack_code<BITS>(w, j);
}

template <int BITS>
__global__ void __launch_bounds__(INF_THREADS, 1)
k_infer_bf16(const __grid_constant__ CUtensorMap tmap_x,      // X [tokens, d_in] bf16, box 64 x 128, swizzled
             const __grid_constant__ CUtensorMap tmap_c,      // codes [d_out, words] uint32, box (4 BITS) x tile_n
             const InferArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* c_base = smem + (size_t)INF_OP_STAGES * INF_OP_BYTES;
  InferBarriers* bars = reinterpret_cast<InferBarriers*>(c_base + (size_t)INF_C_STAGES * INF_C_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = a.tiles_m * a.tiles_n;
  const int N = a.tile_n;
  constexpr int CW = 4 * BITS;                                 // code words per row and k-step (128 codes)
  auto x_tile = [&](int st) { return smem + (size_t)st * INF_OP_BYTES; };
  auto w_tile = [&](int st) { return smem + (size_t)st * INF_OP_BYTES + INF_X_BYTES; };
  auto c_tile = [&](int st) { return c_base + (size_t)st * INF_C_BYTES; };

  if (threadIdx.x == 0) {
    for (int i = 0; i < INF_OP_STAGES; ++i) {
      ptx::mbar_init(&bars->full_x[i], 1);
      ptx::mbar_init(&bars->full_w[i], INF_DEQ_THREADS);
      ptx::mbar_init(&bars->empty_op[i], 1);
    }
    for (int i = 0; i < INF_C_STAGES; ++i) {
      ptx::mbar_init(&bars->full_c[i], 1);
      ptx::mbar_init(&bars->empty_c[i], INF_DEQ_THREADS);
    }
    for (int i = 0; i < INF_ACC; ++i) {
      ptx::mbar_init(&bars->tmem_full[i], 1);
      ptx::mbar_init(&bars->tmem_empty[i], 128);
    }
    bars->abort = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tmap_x);
    ptx::prefetch_tmap(&tmap_c);
  }
  if (warp == 1) {
    ptx::tmem_alloc(&bars->tmem_base, INF_ACC * INF_ACC_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;

  if (warp == 0) {
    // ------------------------------ TMA: X tiles (shallow ring) ------------------------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      for (int t = blockIdx.x; t < num_tiles && !bars->abort; t += gridDim.x) {
        const int m0 = (t / a.tiles_n) * INF_M;
        for (int kb = 0; kb < a.num_kb; ++kb) {      // no flag loads here: see the GEMM producers
          bounded_wait(&bars->empty_op[stage], phase ^ 1, bars);
          // only the rows that hold tokens are copied; the other rows of the operand are never stored
          // from (an MMA output row depends on its own input row only)
          ptx::mbar_arrive_expect_tx(&bars->full_x[stage], (uint32_t)(2 * a.x_rows * 128));
          ptx::tma_load_2d(x_tile(stage), &tmap_x, &bars->full_x[stage], kb * INF_BK, m0);
          ptx::tma_load_2d(x_tile(stage) + INF_X_BYTES / 2, &tmap_x, &bars->full_x[stage], kb * INF_BK + 64, m0);
          if (++stage == INF_OP_STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 2) {
    // ------------------------------ TMA: packed code words (deep ring) ------------------------------
    if (lane == 0) {
      int cs = 0; uint32_t cphase = 0;
      for (int t = blockIdx.x; t < num_tiles && !bars->abort; t += gridDim.x) {
        const int n0 = (t % a.tiles_n) * N;
        for (int kb = 0; kb < a.num_kb; ++kb) {      // no flag loads here: see the GEMM producers
          bounded_wait(&bars->empty_c[cs], cphase ^ 1, bars);
          ptx::mbar_arrive_expect_tx(&bars->full_c[cs], (uint32_t)(N * CW * 4));
          ptx::tma_load_2d(c_tile(cs), &tmap_c, &bars->full_c[cs], kb * CW, n0);
          if (++cs == INF_C_STAGES) { cs = 0; cphase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      const uint32_t idesc = ptx::make_idesc_bf16(INF_M, N, false, false);
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      for (int t = blockIdx.x; t < num_tiles && !bars->abort; t += gridDim.x) {
        bounded_wait(&bars->tmem_empty[acc], acc_phase ^ 1, bars);
        if (bars->abort) break;
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * INF_ACC_COLS);
        for (int kb = 0; kb < a.num_kb; ++kb) {
          bounded_wait(&bars->full_x[stage], phase, bars);
          bounded_wait(&bars->full_w[stage], phase, bars);
          ptx::tc_fence_after_sync();
          const uint32_t xa = ptx::smem_u32(x_tile(stage)), wa = ptx::smem_u32(w_tile(stage));
#pragma unroll
          for (int ks = 0; ks < INF_BK / UMMA_K; ++ks) {     // 8 steps of 16; steps 4..7 are the second 64-wide tile
            const uint64_t da = ptx::make_smem_desc_sw128(xa + (ks >> 2) * (INF_X_BYTES / 2) + (ks & 3) * 32, 16, 1024);
            const uint64_t db = ptx::make_smem_desc_sw128(wa + (ks >> 2) * (INF_W_BYTES / 2) + (ks & 3) * 32, 16, 1024);
            ptx::mma_bf16_ss(d_tmem, da, db, idesc, (kb | ks) != 0 ? 1u : 0u);
          }
          ptx::mma_commit(&bars->empty_op[stage]);
          if (++stage == INF_OP_STAGES) { stage = 0; phase ^= 1; }
        }
        ptx::mma_commit(&bars->tmem_full[acc]);
        if (++acc == INF_ACC) { acc = 0; acc_phase ^= 1; }
      }
    }
    __syncwarp();
  } else if (warp >= 4 && warp < 8) {
    // ------------------------------ epilogue: lane = token ------------------------------
    const int quarter = warp & 3;
    int acc = 0; uint32_t acc_phase = 0;
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
      const int m0 = (t / a.tiles_n) * INF_M, n0 = (t % a.tiles_n) * N;
      bounded_wait(&bars->tmem_full[acc], acc_phase, bars);
      ptx::tc_fence_after_sync();
      const int tok = m0 + quarter * 32 + lane;
      const int nchunks = N >> 4;                              // 16 columns at a time
      for (int c = 0; c < nchunks; ++c) {
        uint32_t raw[16];
        ptx::tmem_ld_32x16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * INF_ACC_COLS + c * 16), raw);
        ptx::tmem_ld_wait();
        if (c == nchunks - 1) {
          ptx::tc_fence_before_sync();
          ptx::mbar_arrive(&bars->tmem_empty[acc]);
        }
        if (tok < a.tokens) {
          __nv_bfloat16* dst = a.Y + (size_t)tok * a.d_out + n0 + c * 16;
#pragma unroll
          for (int v = 0; v < 2; ++v) {
            if (n0 + c * 16 + v * 8 < a.d_out) {
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
      if (++acc == INF_ACC) { acc = 0; acc_phase ^= 1; }
    }
  } else if (warp >= 8) {
    // ------------------------------ dequantizers: thread = (weight row, 32 codes) ------------------------------
    const int pt = threadIdx.x - 256;                          // 0 .. 383
    const int row = pt >> 2, q = pt & 3;                       // row of the tile, 32-code quarter of the k-step
    const bool active = row < N;
    constexpr float kScale = (float)(1 << BITS);
    int stage = 0; uint32_t phase = 0;                         // operand ring
    int cs = 0; uint32_t cphase = 0;                           // code ring
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
      const int n0 = (t % a.tiles_n) * N;
      const int o = n0 + row;
      const bool row_ok = active && o < a.d_out;
      const __half* s_row = a.s16 + (size_t)o * a.ngroups;
      const __half* b_row = a.b16 + (size_t)o * a.ngroups;
      // s, b of the group of this thread's 32 codes (group size is a multiple of 32), fetched one k-step ahead
      auto load_sb = [&](int kb, float& s_, float& b_) {
        const int k = kb * INF_BK + q * 32;
        s_ = 0.f; b_ = 0.f;                                    // rows / columns beyond the weight contribute nothing
        if (row_ok && k < a.d_in) {
          const int g = a.group_shift >= 0 ? (k >> a.group_shift) : (k / a.group);
          s_ = __half2float(__ldg(s_row + g));
          b_ = __half2float(__ldg(b_row + g));
        }
      };
      float s_next, b_next;
      load_sb(0, s_next, b_next);
      for (int kb = 0; kb < a.num_kb; ++kb) {
        const float s2 = s_next * kScale, b2 = b_next - s_next * kScale;     // W_q = m * s2 + b2, m = 1 + u / 2^BITS
        if (kb + 1 < a.num_kb) load_sb(kb + 1, s_next, b_next);
        bounded_wait(&bars->full_c[cs], cphase, bars);         // the code words have landed
        bounded_wait(&bars->empty_op[stage], phase ^ 1, bars); // the operand slot is free (its MMAs completed)
        if (active) {
          const uint8_t* crow = c_tile(cs) + row * (CW * 4) + q * (BITS * 4);
          uint32_t w[BITS];
          if constexpr (BITS == 4) {
            const uint4 v = *reinterpret_cast<const uint4*>(crow);
            w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
          } else {
#pragma unroll
            for (int i = 0; i < BITS; ++i) w[i] = reinterpret_cast<const uint32_t*>(crow)[i];
          }
          float m[32];
          unpack_codes32<BITS>(w, m);
          // W_q = u * s + b (Eq. 9 on the unsigned code) in fp32, rounded to bf16, into the K-major swizzled
          // B operand: 64-k tile q >> 1, 16-byte chunks (q & 1) * 4 .. + 3 of row `row`
          uint8_t* wrow = w_tile(stage) + (q >> 1) * (INF_W_BYTES / 2) + row * 128;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint4 o4;
            o4.x = pack_bf16x2(fmaf(m[c * 8 + 0], s2, b2), fmaf(m[c * 8 + 1], s2, b2));
            o4.y = pack_bf16x2(fmaf(m[c * 8 + 2], s2, b2), fmaf(m[c * 8 + 3], s2, b2));
            o4.z = pack_bf16x2(fmaf(m[c * 8 + 4], s2, b2), fmaf(m[c * 8 + 5], s2, b2));
            o4.w = pack_bf16x2(fmaf(m[c * 8 + 6], s2, b2), fmaf(m[c * 8 + 7], s2, b2));
            *reinterpret_cast<uint4*>(wrow + ((((q & 1) * 4 + c) ^ (row & 7)) << 4)) = o4;
          }
        }
        ptx::mbar_arrive(&bars->empty_c[cs]);                  // code words consumed
        ptx::fence_proxy_async_smem();                         // the operand is read by the tensor cores
        ptx::mbar_arrive(&bars->full_w[stage]);
        if (++stage == INF_OP_STAGES) { stage = 0; phase ^= 1; }
        if (++cs == INF_C_STAGES) { cs = 0; cphase ^= 1; }
      }
    }
  }

  // ------------------------------ teardown ------------------------------
  if (bars->abort) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);            // let copies in flight land before shared memory is released
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, INF_ACC * INF_ACC_COLS);
  }
}

// ---------------------------------------------------------------------------
// One or two tokens: a plain-ALU matrix-vector kernel.  With so few tokens there is nothing for the tensor
// cores to amortise (an MMA has a fixed cost per 16 values of k), while 1 + tokens FMAs per weight keep the
// FP32 pipe below the time the packed weight needs to arrive from HBM.
//   * X is copied to shared memory once per CTA as fp32, together with the sum of each 32-value piece;
//   * a warp owns GEMV_ROWS weight rows at a time and walks along k; a lane takes 32 codes of each row
//     (16 or 12 contiguous bytes: the warp reads 512 / 384 contiguous bytes per row) and the matching 32
//     values of X, so the reads of X are shared by the rows;
//   * codes become m = 1 + u / 2^bits (unpack_codes32); per piece  sum x W_q = (2^bits s) sum x m + (b - 2^bits s) sum x.
// ---------------------------------------------------------------------------
constexpr int GEMV_ROWS = 2;
constexpr int GEMV_THREADS = 256;

template <int BITS, int TOK>
__global__ void __launch_bounds__(GEMV_THREADS)
k_infer_gemv(const __nv_bfloat16* __restrict__ X, const uint32_t* __restrict__ codes, const __half* __restrict__ s16,
             const __half* __restrict__ b16, __nv_bfloat16* __restrict__ Y, int d_in, int d_out, int group_shift,
             int group, int ngroups) {
  extern __shared__ __align__(16) float gemv_smem[];
  const int units = d_in >> 5;                                  // 32-code pieces per row
  // X in shared memory as [token][v = 0..7][unit][4]: value k = 32 unit + 4 v + e of a token.  A lane owns a
  // unit, so for a fixed v the 32 lanes of a warp read 32 consecutive float4 (no bank conflicts); with the
  // natural [token][k] layout their float4 would be 128 bytes apart and hit the same four banks.
  float* xs = gemv_smem;
  float* xsum = gemv_smem + (size_t)TOK * d_in;                 // [TOK][units]
  for (int i = threadIdx.x; i < TOK * d_in; i += GEMV_THREADS) {
    const int t = i / d_in, k = i - t * d_in;
    xs[(size_t)t * d_in + ((size_t)((k >> 2) & 7) * units + (k >> 5)) * 4 + (k & 3)] = __bfloat162float(X[i]);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < TOK * units; i += GEMV_THREADS) {
    const int t = i / units, u = i - t * units;
    float a = 0.f;
#pragma unroll
    for (int v = 0; v < 8; ++v) {
      const float4 x4 = *reinterpret_cast<const float4*>(xs + (size_t)t * d_in + ((size_t)v * units + u) * 4);
      a += (x4.x + x4.y) + (x4.z + x4.w);
    }
    xsum[i] = a;
  }
  __syncthreads();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int warps_total = gridDim.x * (GEMV_THREADS / 32);
  const int row_words = (d_in * BITS) >> 5;
  constexpr float kScale = (float)(1 << BITS);
  for (int r0 = (blockIdx.x * (GEMV_THREADS / 32) + warp) * GEMV_ROWS; r0 < d_out; r0 += warps_total * GEMV_ROWS) {
    float acc[GEMV_ROWS][TOK];
#pragma unroll
    for (int r = 0; r < GEMV_ROWS; ++r)
#pragma unroll
      for (int t = 0; t < TOK; ++t) acc[r][t] = 0.f;
    for (int u = lane; u < units; u += 32) {
      const int g = group_shift >= 0 ? ((u << 5) >> group_shift) : ((u << 5) / group);
      float dot[GEMV_ROWS][TOK];
#pragma unroll
      for (int r = 0; r < GEMV_ROWS; ++r)
#pragma unroll
        for (int t = 0; t < TOK; ++t) dot[r][t] = 0.f;
      uint32_t w[GEMV_ROWS][BITS];
#pragma unroll
      for (int r = 0; r < GEMV_ROWS; ++r) {
        const int row = min(r0 + r, d_out - 1);                 // rows beyond the weight repeat the last one, unused
        const uint32_t* src = codes + (size_t)row * row_words + (size_t)u * BITS;
        if constexpr (BITS == 4) {
          const uint4 v = __ldg(reinterpret_cast<const uint4*>(src));
          w[r][0] = v.x; w[r][1] = v.y; w[r][2] = v.z; w[r][3] = v.w;
        } else {
#pragma unroll
          for (int i = 0; i < BITS; ++i) w[r][i] = __ldg(src + i);
        }
      }
#pragma unroll
      for (int v = 0; v < 8; ++v) {                             // 4 values of k at a time: x of every token, code of every row
        float4 x4[TOK];
#pragma unroll
        for (int t = 0; t < TOK; ++t)
          x4[t] = *reinterpret_cast<const float4*>(xs + (size_t)t * d_in + ((size_t)v * units + u) * 4);
#pragma unroll
        for (int r = 0; r < GEMV_ROWS; ++r) {
          const float m0 = unpack_code<BITS>(w[r], v * 4 + 0), m1 = unpack_code<BITS>(w[r], v * 4 + 1);
          const float m2 = unpack_code<BITS>(w[r], v * 4 + 2), m3 = unpack_code<BITS>(w[r], v * 4 + 3);
#pragma unroll
          for (int t = 0; t < TOK; ++t) {
            dot[r][t] = fmaf(x4[t].x, m0, dot[r][t]);
            dot[r][t] = fmaf(x4[t].y, m1, dot[r][t]);
            dot[r][t] = fmaf(x4[t].z, m2, dot[r][t]);
            dot[r][t] = fmaf(x4[t].w, m3, dot[r][t]);
          }
        }
      }
#pragma unroll
      for (int r = 0; r < GEMV_ROWS; ++r) {
        const int row = min(r0 + r, d_out - 1);
        const float s_ = __half2float(__ldg(s16 + (size_t)row * ngroups + g));
        const float b_ = __half2float(__ldg(b16 + (size_t)row * ngroups + g));
        const float s2 = s_ * kScale, b2 = b_ - s2;
#pragma unroll
        for (int t = 0; t < TOK; ++t) acc[r][t] += fmaf(s2, dot[r][t], b2 * xsum[t * units + u]);
      }
    }
#pragma unroll
    for (int r = 0; r < GEMV_ROWS; ++r)
#pragma unroll
      for (int t = 0; t < TOK; ++t) {
        float v = acc[r][t];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        if (lane == 0 && r0 + r < d_out) Y[(size_t)t * d_out + r0 + r] = __float2bfloat16_rn(v);
      }
  }
}

inline size_t gemv_smem_bytes(int tokens, int d_in) { return (size_t)tokens * (d_in + (d_in >> 5)) * sizeof(float); }

inline bool gemv_supported(const Params& p) {
  return p.tokens <= 2 && p.d_in % 32 == 0     // measured: beyond two tokens the tensor-core kernel is the faster one
         && gemv_smem_bytes(p.tokens, p.d_in) <= 200 * 1024;
}

inline l4q_status launch_infer_gemv(const Params& p, const void* X, const uint32_t* codes, const __half* s16,
                                    const __half* b16, void* Y, cudaStream_t st) {
  int shift = -1;
  for (int sh = 5; sh < 31; ++sh)
    if ((1 << sh) == p.group) shift = sh;
  const size_t smem = gemv_smem_bytes(p.tokens, p.d_in);
  const int quads = ceil_div(p.d_out, GEMV_ROWS);
  // several CTAs per SM (registers and shared memory permitting): more loads in flight, finer balance
  const int per_sm = std::max(1, std::min(6, (int)((200 * 1024) / std::max<size_t>(smem, 1))));
  const int grid = std::min(ceil_div(quads, GEMV_THREADS / 32), sm_count() * per_sm);
  auto launch = [&](auto kern) -> l4q_status {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return cuda_fail();
    kern<<<grid, GEMV_THREADS, smem, st>>>(reinterpret_cast<const __nv_bfloat16*>(X), codes, s16, b16,
                                           reinterpret_cast<__nv_bfloat16*>(Y), p.d_in, p.d_out, shift, p.group, p.ngroups);
    return cudaGetLastError() == cudaSuccess ? L4Q_OK : L4Q_ERR_CUDA;
  };
  const int key = p.bits * 10 + p.tokens;
  switch (key) {
    case 41: return launch(k_infer_gemv<4, 1>);
    case 42: return launch(k_infer_gemv<4, 2>);
    case 31: return launch(k_infer_gemv<3, 1>);
    case 32: return launch(k_infer_gemv<3, 2>);
    default: return L4Q_ERR_UNSUPPORTED;
  }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------

inline bool infer_supported(const Params& p) {
  if (p.bits != 3 && p.bits != 4) return false;
  if (p.group % 32 != 0) return false;                          // a unit's 32 codes share one group
  const long long bits_per_row = (long long)p.d_in * p.bits;
  if (bits_per_row % 32 != 0 || ((bits_per_row / 32) * 4) % 16 != 0) return false;   // TMA row pitch of the codes
  return true;
}

// Weight rows per tile: the multiple of 16 (<= INF_NMAX) for which the busiest SM gets the fewest rows.
inline int infer_pick_tile_n(int d_out, int tiles_m, int sms) {
  int best = 16; long long best_cost = -1;
  for (int n = 16; n <= INF_NMAX; n += 16) {
    const long long tiles = (long long)tiles_m * ceil_div(d_out, n);
    const long long cost = ((tiles + sms - 1) / sms) * n;       // rows of W the busiest SM dequantizes per token tile
    if (best_cost < 0 || cost < best_cost || (cost == best_cost && n > best)) { best = n; best_cost = cost; }
  }
  return best;
}

inline l4q_status launch_infer_bf16(const Params& p, const void* X, const uint32_t* codes, const __half* s16,
                                    const __half* b16, void* Y, cudaStream_t st) {
  InferArgs a{};
  a.tokens = p.tokens; a.d_in = p.d_in; a.d_out = p.d_out; a.bits = p.bits; a.group = p.group; a.ngroups = p.ngroups;
  a.tiles_m = ceil_div(p.tokens, INF_M);
  a.tile_n = infer_pick_tile_n(p.d_out, a.tiles_m, sm_count());
  a.tiles_n = ceil_div(p.d_out, a.tile_n);
  a.num_kb = ceil_div(p.d_in, INF_BK);
  a.group_shift = -1;
  for (int sh = 5; sh < 31; ++sh)
    if ((1 << sh) == p.group) a.group_shift = sh;
  a.s16 = s16; a.b16 = b16;
  a.Y = reinterpret_cast<__nv_bfloat16*>(Y);
  CUtensorMap tx, tc;
  a.x_rows = std::min(INF_M, (p.tokens + 7) / 8 * 8);
  if (!make_tmap_bf16(&tx, X, p.tokens, p.d_in, a.x_rows)) return cuda_fail();
  if (!make_tmap_words(&tc, codes, p.d_out, ((uint64_t)p.d_in * p.bits) >> 5, 4 * p.bits, a.tile_n)) return cuda_fail();
  const size_t smem = infer_smem_bytes();
  const int grid = std::min(a.tiles_m * a.tiles_n, sm_count());
  auto launch = [&](auto kern) -> l4q_status {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return cuda_fail();
    kern<<<grid, INF_THREADS, smem, st>>>(tx, tc, a);
    return cudaGetLastError() == cudaSuccess ? L4Q_OK : L4Q_ERR_CUDA;
  };
  return p.bits == 4 ? launch(k_infer_bf16<4>) : launch(k_infer_bf16<3>);
}

}  // namespace l4q
