// Fully quantized inference (Sec. 3.2, App. F): Y = X W_q^T where only the export of l4q_pack_int is
// kept -- bit-packed unsigned codes u and one fp16 scale / offset per group, W_q = u * s16 + b16.
//
// The regime of the paper's deployment measurements is a handful of tokens per step (batch 1..64), so the
// kernel is bound by reading the packed weight once (bits/8 bytes per weight) and by turning it into bf16,
// and is built around that:
//   * tokens are the MMA's M (one 128-row tile; only the rows that hold tokens are loaded), output features
//     its N, in tiles of 16..128 rows of W chosen so that the tiles fill the SMs evenly;
//   * the packed code words of a tile (N rows x 64 or 48 bytes per 128-deep k-step) arrive by TMA through a
//     deep ring (8 steps in flight: they are the only HBM traffic), the X tile (128-byte-swizzled, from L2)
//     and the dequantized operand through a ring of as many steps as shared memory holds (up to 6);
//   * 16 dequantizer warps: a warp takes one block of 16 weight rows x 128 k at a time (thread = one row and
//     two runs of 32 codes), the blocks of consecutive k-steps going round the warps, so that all of them stay
//     busy whatever N is and several k-steps are being dequantized at once.  Codes become bf16
//     W_q = u * s + b with fp32 arithmetic and are written as the MMA's B operand in
//     the swizzled K-major layout; one thread issues tcgen05.mma (bf16 x bf16 -> fp32 in tensor memory);
//   * warps 4..7 drain the 128 x N accumulator when a tile's k loop is done.
// Roles (640 threads): warp 0 = TMA of X, warp 2 = TMA of the code words, warps 1 and 3 = MMA issuers (1 owns TMEM),
// warps 4..19 = dequantizers.  Every mbarrier wait is bounded (bounded_wait).
#pragma once

#include "l4q_common.cuh"
#include "l4q_gemm.cuh"
#include "l4q_ptx.cuh"
#include "l4q_wtile.cuh"

namespace l4q {

constexpr int INF_M = 128;                 // tokens per tile (MMA M)
constexpr int INF_NMAX = 128;              // most weight rows per tile (MMA N, a multiple of 16 chosen per problem)
constexpr int INF_BK = 128;                // k per pipeline step
constexpr int INF_MAX_OP_STAGES = 6;       // X tile + dequantized W tile
constexpr int INF_C_STAGES = 8;            // packed code words, loaded far ahead: they are what comes from HBM
constexpr int INF_THREADS = 640;
constexpr int INF_WORKERS = 16;            // dequantizer warps (4..19)
constexpr int INF_ACC = 2;
constexpr int INF_HALF_COLS = 128;         // TMEM columns of one issuer's half of an accumulator stage
constexpr int INF_ACC_COLS = 2 * INF_HALF_COLS;

struct InferArgs {
  int tokens, d_in, d_out, bits, group, ngroups;
  int tile_n;                              // weight rows per tile
  int nb;                                  // tile_n / 16: blocks of 16 rows per k-step
  int group_shift;                         // log2(group size) if it is a power of two, else -1
  int x_rows;                              // token rows a TMA box of X brings in (8 .. 128)
  int tiles_m, tiles_n, num_kb;
  int op_stages;                           // depth of the operand ring
  int one_group;                           // group size is a multiple of 128: a k-step lies in one group
  int workers;                             // dequantizer warps at work: min(INF_WORKERS, nb * op_stages)
  uint32_t x_bytes, w_bytes, c_bytes;      // per stage: X tile (two boxes of x_rows x 64), W tile (two of N x 64), codes
  const __half *s16, *b16;
  __nv_bfloat16* Y;
};

struct __align__(8) InferBarriers {
  uint64_t full_op[INF_MAX_OP_STAGES];     // the X tile has landed and the dequantized B operand of the stage is complete
  uint64_t empty_op[INF_MAX_OP_STAGES];    // the MMAs reading the operand stage have completed
  uint64_t full_c[INF_C_STAGES];           // code words have landed
  uint64_t empty_c[INF_C_STAGES];          // the dequantizers have read the code words
  uint64_t tmem_full[INF_ACC], tmem_empty[INF_ACC];
  uint32_t tmem_base;
  volatile uint32_t abort;
};

constexpr size_t INF_SMEM_LIMIT = 227 * 1024;

// (a & b) | c in one logic instruction, all three operands in registers.
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// 32 unsigned codes of one weight row (starting at a multiple of 32 codes of the LSB-first bitstream), each
// returned as the float m = 1 + u / 2^BITS: the code is moved into the top mantissa bits under the exponent
// of 1.0 (one shift and one logic op, no integer-to-float conversion).  The caller folds the affine map back:
// u * s + b = m * (2^BITS s) + (b - 2^BITS s), a single fma.
template <int BITS>
__device__ __forceinline__ float unpack_code(const uint32_t (&w)[BITS], int j, uint32_t mask, uint32_t one) {   // j: compile-time after unrolling
  constexpr int POS = 23 - BITS;                               // bit position of the code inside the mantissa
  const int bit = j * BITS, wd = bit >> 5, off = bit & 31;
  uint32_t v;
  if (off + BITS > 32) v = __funnelshift_r(w[wd], w[wd + 1 < BITS ? wd + 1 : wd], off) << POS;   // code straddles two words
  else v = (off <= POS) ? (w[wd] << (POS - off)) : (w[wd] >> (off - POS));
  return __uint_as_float(and_or(v, mask, one));
}

// The mask of the code field and the exponent of 1.0 for unpack_code, in registers that the compiler cannot fold
// back into immediates (with two immediates the and-or takes two instructions).
template <int BITS>
__device__ __forceinline__ void unpack_constants(uint32_t& mask, uint32_t& one) {
  mask = ((1u << BITS) - 1u) << (23 - BITS);
  one = 0x3F800000u;
  asm volatile("" : "+r"(mask), "+r"(one));
}

// 32 codes of one weight row -> 16 words of bf16 pairs W_q = u * s + b (Eq. 9 on the unsigned code), formed in
// fp32 and rounded once.  The bitstream is cut into windows of 12 bits (3 or 4 codes); one funnel shift puts a
// window at mantissa bits 11..22, so that a code at bit position p reads, with the exponent of 1.0 or-ed in, as
// m = 1 + u 2^(p-23), and u s + b = m S_p + (b - S_p) with S_p = s 2^(23-p): one logic op and one fma
// per code, with three or four (S_p, b - S_p) pairs per thread.  S_p <= 2^12 s, so b - S_p is exact to
// 2^-12 of a quantization step.
template <int BITS>
__device__ __forceinline__ void dequant_codes32(const uint32_t (&w)[BITS], float s, float b, uint32_t (&out)[16]) {
  constexpr int CPW = 12 / BITS;                               // codes per window
  constexpr uint32_t MASK = (1u << BITS) - 1u;
  float S[CPW], C[CPW];
  uint32_t mask[CPW];
  // the masks and the exponent of 1.0 are kept in registers (opaque to the compiler), so that a code costs one
  // three-input logic instruction; written as immediates they cost two
  uint32_t one = 0x3F800000u;
  asm volatile("" : "+r"(one));
#pragma unroll
  for (int i = 0; i < CPW; ++i) {
    S[i] = s * (float)(1 << (12 - BITS * i));                  // 2^(23 - p), p = 11 + BITS i
    C[i] = b - S[i];
    mask[i] = MASK << (11 + BITS * i);
    asm volatile("" : "+r"(mask[i]));
  }
  constexpr int NWIN = (32 + CPW - 1) / CPW;
  uint32_t win[NWIN];
#pragma unroll
  for (int v = 0; v < NWIN; ++v) {
    if (v == 0) {
      win[v] = w[0] << 11;
    } else {
      const int sh = 12 * v - 11, wd = sh >> 5, off = sh & 31;
      win[v] = __funnelshift_r(w[wd], wd + 1 < BITS ? w[wd + 1] : 0u, off);
    }
  }
#pragma unroll
  for (int c = 0; c < 32; c += 2) {
    const int v0 = c / CPW, i0 = c % CPW, v1 = (c + 1) / CPW, i1 = (c + 1) % CPW;
    const float m0 = __uint_as_float(and_or(win[v0], mask[i0], one));
    const float m1 = __uint_as_float(and_or(win[v1], mask[i1], one));
    out[c >> 1] = pack_bf16x2(fmaf(m0, S[i0], C[i0]), fmaf(m1, S[i1], C[i1]));
  }
}

template <int BITS>
__global__ void __launch_bounds__(INF_THREADS, 1)
k_infer_bf16(const __grid_constant__ CUtensorMap tmap_x,      // X [tokens, d_in] bf16, box 64 x x_rows, swizzled
             const __grid_constant__ CUtensorMap tmap_c,      // codes [d_out, words] uint32, box (4 BITS) x tile_n
             const InferArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t op_bytes = a.x_bytes + a.w_bytes;
  const int S = a.op_stages;
  uint8_t* c_base = smem + (size_t)S * op_bytes;
  InferBarriers* bars = reinterpret_cast<InferBarriers*>(c_base + (size_t)INF_C_STAGES * a.c_bytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = a.tiles_m * a.tiles_n;
  const int N = a.tile_n, NB = a.nb;
  constexpr int CW = 4 * BITS;                                 // code words per row and k-step (128 codes)
  auto x_tile = [&](int st) { return smem + (size_t)st * op_bytes; };
  auto w_tile = [&](int st) { return smem + (size_t)st * op_bytes + a.x_bytes; };
  auto c_tile = [&](int st) { return c_base + (size_t)st * a.c_bytes; };

  if (threadIdx.x == 0) {
    for (int i = 0; i < S; ++i) {
      ptx::mbar_init(&bars->full_op[i], (uint32_t)(NB * 32 + 1));
      ptx::mbar_init(&bars->empty_op[i], 1);
    }
    for (int i = 0; i < INF_C_STAGES; ++i) {
      ptx::mbar_init(&bars->full_c[i], 1);
      ptx::mbar_init(&bars->empty_c[i], (uint32_t)(NB * 32));
    }
    for (int i = 0; i < INF_ACC; ++i) {
      ptx::mbar_init(&bars->tmem_full[i], 2);
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
    // ------------------------------ TMA: X tiles ------------------------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      for (int t = blockIdx.x; t < num_tiles && !bars->abort; t += gridDim.x) {
        const int m0 = (t / a.tiles_n) * INF_M;
        for (int kb = 0; kb < a.num_kb; ++kb) {      // no flag loads here: see the GEMM producers
          bounded_wait_relaxed(&bars->empty_op[stage], phase ^ 1, bars);
          // only the rows that hold tokens are copied; the other rows of the operand hold whatever the ring
          // held before (an MMA output row depends on its own input row only, and they are never stored)
          ptx::mbar_arrive_expect_tx(&bars->full_op[stage], a.x_bytes);
          ptx::tma_load_2d(x_tile(stage), &tmap_x, &bars->full_op[stage], kb * INF_BK, m0);
          ptx::tma_load_2d(x_tile(stage) + a.x_bytes / 2, &tmap_x, &bars->full_op[stage], kb * INF_BK + 64, m0);
          if (++stage == S) { stage = 0; phase ^= 1; }
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
          bounded_wait_relaxed(&bars->empty_c[cs], cphase ^ 1, bars);
          ptx::mbar_arrive_expect_tx(&bars->full_c[cs], (uint32_t)(N * CW * 4));
          ptx::tma_load_2d(c_tile(cs), &tmap_c, &bars->full_c[cs], kb * CW, n0);
          if (++cs == INF_C_STAGES) { cs = 0; cphase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1 || warp == 3) {
    // ------------------------------ MMA issuers ------------------------------
    // Two threads on two warp schedulers: issuer i takes the k-steps whose running number (over all tiles of the
    // CTA) is i modulo 2 and accumulates them into its own half of the accumulator stage; the epilogue adds the
    // halves.  One thread alone, sharing its scheduler with four busy dequantizer warps, needed 650..900 cycles
    // to issue the eight MMAs of a k-step that execute in about 420.
    if (lane == 0) {
      const int me = warp >> 1;                                // 0 or 1
      const uint32_t idesc = ptx::make_idesc_bf16(INF_M, N, false, false);
      // Descriptors differ in the start-address field only (16-byte units in the low word; shared memory is
      // < 256 KB, so sums never leave the field): the eight offsets of a k-step are kept in registers.
      const uint64_t dx0 = ptx::make_smem_desc_sw128(ptx::smem_u32(smem), 16, 1024);
      const uint64_t dw0 = ptx::make_smem_desc_sw128(ptx::smem_u32(smem) + a.x_bytes, 16, 1024);
      const uint32_t d_hi = (uint32_t)(dx0 >> 32);             // same for both operands
      uint32_t ox[INF_BK / UMMA_K], ow[INF_BK / UMMA_K];
#pragma unroll
      for (int ks = 0; ks < INF_BK / UMMA_K; ++ks) {           // steps 4..7 are the second 64-wide tile
        ox[ks] = (uint32_t)dx0 + (uint32_t)((ks >> 2) * (a.x_bytes >> 5) + (ks & 3) * 2);
        ow[ks] = (uint32_t)dw0 + (uint32_t)((ks >> 2) * (a.w_bytes >> 5) + (ks & 3) * 2);
      }
      const uint32_t step = op_bytes >> 4;
      const uint32_t full_op_a = ptx::smem_u32(&bars->full_op[0]);
      // this issuer's next k-step: number within the tile, ring stage and phase (S >= 2)
      int kb = me, stage = me; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      for (int t = blockIdx.x; t < num_tiles && !bars->abort; t += gridDim.x) {
        bounded_wait(&bars->tmem_empty[acc], acc_phase ^ 1, bars);
        if (bars->abort) break;
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * INF_ACC_COLS + me * INF_HALF_COLS);
        uint32_t accumulate = 0;
        for (; kb < a.num_kb; kb += 2) {
          bounded_wait_a(full_op_a + (uint32_t)stage * 8u, phase, bars);
          ptx::tc_fence_after_sync();
          const uint32_t so = (uint32_t)stage * step;
#pragma unroll
          for (int ks = 0; ks < INF_BK / UMMA_K; ++ks) {
            const uint64_t da = ((uint64_t)d_hi << 32) | (uint64_t)(ox[ks] + so);
            const uint64_t db = ((uint64_t)d_hi << 32) | (uint64_t)(ow[ks] + so);
            ptx::mma_bf16_ss(d_tmem, da, db, idesc, ks != 0 ? 1u : accumulate);
          }
          accumulate = 1;
          ptx::mma_commit(&bars->empty_op[stage]);
          stage += 2;
          if (stage >= S) { stage -= S; phase ^= 1; }
        }
        kb -= a.num_kb;                                        // the same k-step, counted within the next tile
        if (accumulate) ptx::mma_commit(&bars->tmem_full[acc]);
        else ptx::mbar_arrive(&bars->tmem_full[acc]);          // (a one-step tile: nothing from this issuer)
        if (++acc == INF_ACC) { acc = 0; acc_phase ^= 1; }
      }
    }
    __syncwarp();
  } else if (warp >= 4) {
    // ------------------------------ dequantizers: warp = block of 16 rows x 128 k, thread = (row, 2 x 32 codes) ----
    const int worker = warp - 4;                               // 0 .. 15
    // Row of the block and the two 32-code quarters of the k-step a thread takes.  The eight lanes that one
    // shared-memory wavefront serves hold eight different rows, each with quarter (row / 2 + j) % 4: their 16-byte
    // loads of the code words fall into eight different bank groups, and so do their stores into the swizzled
    // operand (chunk ((q & 1) * 4 + c) ^ (row % 8)).  The second quarter is two further on.
    const int r16 = (lane >> 4) * 8 + (lane & 7);
    const int q0 = (((lane & 7) >> 1) + ((lane >> 3) & 1)) & 3;
    const int quarter = warp & 3;                              // epilogue (warps 4..7): TMEM lane quarter
    const uint32_t smem_a = ptx::smem_u32(smem);
    const uint32_t c_base_a = smem_a + (uint32_t)S * op_bytes;
    const uint32_t full_c_a = ptx::smem_u32(&bars->full_c[0]), empty_c_a = ptx::smem_u32(&bars->empty_c[0]);
    const uint32_t full_op_a = ptx::smem_u32(&bars->full_op[0]), empty_op_a = ptx::smem_u32(&bars->empty_op[0]);
    // byte offsets of this thread inside a block of 16 rows: its two runs of code words, and the eight 16-byte
    // chunks it stores (the swizzle term row % 8 does not depend on the block)
    const uint32_t c_off[2] = {(uint32_t)(r16 * (CW * 4) + q0 * (BITS * 4)), (uint32_t)(r16 * (CW * 4) + (q0 ^ 2) * (BITS * 4))};
    uint32_t w_off[2][4];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int q = q0 ^ (h * 2);
#pragma unroll
      for (int c = 0; c < 4; ++c)
        w_off[h][c] = (uint32_t)(q >> 1) * (a.w_bytes / 2) + (uint32_t)(r16 * 128) +
                      ((((uint32_t)((q & 1) * 4 + c)) ^ (uint32_t)(r16 & 7)) << 4);
    }
    int stage = 0; uint32_t phase = 0;                         // operand ring, at k-step `ks` of the current tile
    int cs = 0; uint32_t cphase = 0;                           // code ring
    auto advance = [&](int d) {
      stage += d; while (stage >= S) { stage -= S; phase ^= 1; }
      cs += d; while (cs >= INF_C_STAGES) { cs -= INF_C_STAGES; cphase ^= 1; }
    };
    int acc = 0; uint32_t acc_phase = 0;
    uint32_t tiles_done = 0;                                   // tiles of this CTA so far (epilogue warps)
    // The warps at work together span ceil(workers / NB) k-steps.  A wait on a ring barrier tells phases apart by
    // parity only, so a warp must never be two laps of a ring ahead of it: the span may not exceed the depth of
    // either ring, which is what limits the number of warps at work when N is small (the others only idle).
    const bool works = worker < a.workers;
    // from one block to the warp's next: a.workers blocks further on
    const int step_ks = a.workers / NB, step_blk = a.workers - step_ks * NB;
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
      const int m0 = (t / a.tiles_n) * INF_M, n0 = (t % a.tiles_n) * N;
      int ks = works ? 0 : a.num_kb, blk = worker;
      while (works && blk >= NB) { blk -= NB; ++ks; }
      advance(min(ks, a.num_kb));                            // (a warp without a block in this tile just moves on)
      // s, b (fp16 bit patterns) of the groups of this thread's codes (group size is a multiple of 32), for quarter
      // q0 and for quarter q0 ^ 2, fetched one block ahead and left untouched in registers until they are used.
      // When the group size is a multiple of 128 both quarters lie in one group.
      auto load_sb = [&](int ks_, int blk_, uint32_t (&sv)[2], uint32_t (&bv)[2]) {
        const int o = n0 + blk_ * 16 + r16;
        sv[0] = sv[1] = bv[0] = bv[1] = 0u;                    // rows / columns beyond the weight contribute nothing
        if (ks_ < a.num_kb && o < a.d_out) {
          const unsigned short* s_row = reinterpret_cast<const unsigned short*>(a.s16) + (size_t)o * a.ngroups;
          const unsigned short* b_row = reinterpret_cast<const unsigned short*>(a.b16) + (size_t)o * a.ngroups;
          if (a.one_group) {
            const int k = ks_ * INF_BK;
            if (k < a.d_in) {
              const int g = a.group_shift >= 0 ? (k >> a.group_shift) : (k / a.group);
              sv[0] = sv[1] = ptx::ldg_u16(s_row + g);
              bv[0] = bv[1] = ptx::ldg_u16(b_row + g);
            }
          } else {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const int k = ks_ * INF_BK + (q0 ^ (h * 2)) * 32;
              if (k < a.d_in) {
                const int g = a.group_shift >= 0 ? (k >> a.group_shift) : (k / a.group);
                sv[h] = ptx::ldg_u16(s_row + g);
                bv[h] = ptx::ldg_u16(b_row + g);
              }
            }
          }
        }
      };
      uint32_t s_next[2], b_next[2];
      load_sb(ks, blk, s_next, b_next);
      while (ks < a.num_kb) {
        const uint32_t s_cur[2] = {s_next[0], s_next[1]}, b_cur[2] = {b_next[0], b_next[1]};
        int nblk = blk + step_blk, d = step_ks;
        if (nblk >= NB) { nblk -= NB; ++d; }
        load_sb(ks + d, nblk, s_next, b_next);
        bounded_wait_a(full_c_a + (uint32_t)cs * 8u, cphase, bars);          // the code words have landed
        bounded_wait_a(empty_op_a + (uint32_t)stage * 8u, phase ^ 1, bars);  // the operand slot is free (its MMAs completed)
        const uint32_t c_row = c_base_a + (uint32_t)cs * a.c_bytes + (uint32_t)(blk * (16 * CW * 4));
        const uint32_t w_row = smem_a + (uint32_t)stage * op_bytes + a.x_bytes + (uint32_t)(blk * (16 * 128));
        uint32_t w[2][BITS];
#pragma unroll
        for (int h = 0; h < 2; ++h) {                          // (both loads first: they are independent of the stores below)
          const uint32_t at = c_row + c_off[h];
          if constexpr (BITS == 4) {
            const uint4 v = ptx::lds128(at);
            w[h][0] = v.x; w[h][1] = v.y; w[h][2] = v.z; w[h][3] = v.w;
          } else {
#pragma unroll
            for (int i = 0; i < BITS; ++i) w[h][i] = ptx::lds32(at + (uint32_t)(i * 4));
          }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float s_ = __half2float(__ushort_as_half((unsigned short)s_cur[h]));
          const float b_ = __half2float(__ushort_as_half((unsigned short)b_cur[h]));
          uint32_t wv[16];
          dequant_codes32<BITS>(w[h], s_, b_, wv);
          // into the K-major swizzled B operand: 64-k tile q >> 1, 16-byte chunks (q & 1) * 4 .. + 3 of the row
#pragma unroll
          for (int c = 0; c < 4; ++c)
            ptx::sts128(w_row + w_off[h][c], wv[c * 4 + 0], wv[c * 4 + 1], wv[c * 4 + 2], wv[c * 4 + 3]);
        }
        ptx::mbar_arrive_a(empty_c_a + (uint32_t)cs * 8u);     // code words consumed
        ptx::fence_proxy_async_smem();                         // the operand is read by the tensor cores
        ptx::mbar_arrive_a(full_op_a + (uint32_t)stage * 8u);
        blk = nblk;
        if (ks + d < a.num_kb) advance(d);
        else advance(a.num_kb - ks);                           // on to k-step 0 of the CTA's next tile
        ks += d;
      }
      if (warp < 8) {
        // ------------------------------ epilogue: lane = token ------------------------------
        bounded_wait_relaxed(&bars->tmem_full[acc], acc_phase, bars, 512);
        ptx::tc_fence_after_sync();
        const int tok = m0 + quarter * 32 + lane;
        const int nchunks = N >> 3;                            // 8 columns at a time
        // which halves hold a sum: both, unless the tile is a single k-step (then only its issuer's)
        const bool one_step = a.num_kb == 1;
        const int only = one_step ? (int)(tiles_done & 1u) : 0;
        for (int c = 0; c < nchunks; ++c) {
          uint32_t raw[8], raw2[8];
          const uint32_t col = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * INF_ACC_COLS + c * 8);
          ptx::tmem_ld_32x8(col + (uint32_t)(only * INF_HALF_COLS), raw);
          if (!one_step) ptx::tmem_ld_32x8(col + INF_HALF_COLS, raw2);
          ptx::tmem_ld_wait();
          if (c == nchunks - 1) {
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&bars->tmem_empty[acc]);
          }
          if (!one_step) {
#pragma unroll
            for (int i = 0; i < 8; ++i) raw[i] = __float_as_uint(__uint_as_float(raw[i]) + __uint_as_float(raw2[i]));
          }
          if (tok < a.tokens && n0 + c * 8 < a.d_out) {
            uint4 o4;
            o4.x = pack_bf16x2(__uint_as_float(raw[0]), __uint_as_float(raw[1]));
            o4.y = pack_bf16x2(__uint_as_float(raw[2]), __uint_as_float(raw[3]));
            o4.z = pack_bf16x2(__uint_as_float(raw[4]), __uint_as_float(raw[5]));
            o4.w = pack_bf16x2(__uint_as_float(raw[6]), __uint_as_float(raw[7]));
            *reinterpret_cast<uint4*>(a.Y + (size_t)tok * a.d_out + n0 + c * 8) = o4;
          }
        }
        ++tiles_done;
        if (++acc == INF_ACC) { acc = 0; acc_phase ^= 1; }
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
//   * codes become m = 1 + u / 2^bits (unpack_code); per piece  sum x W_q = (2^bits s) sum x m + (b - 2^bits s) sum x.
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
  uint32_t cmask, cone;
  unpack_constants<BITS>(cmask, cone);
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
          const float m0 = unpack_code<BITS>(w[r], v * 4 + 0, cmask, cone), m1 = unpack_code<BITS>(w[r], v * 4 + 1, cmask, cone);
          const float m2 = unpack_code<BITS>(w[r], v * 4 + 2, cmask, cone), m3 = unpack_code<BITS>(w[r], v * 4 + 3, cmask, cone);
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

inline int infer_pick_tile_n(int d_out, int tiles_m, int sms);

// Measured (weights from HBM): at one token the matrix-vector kernel is the faster one on every layer shape; at two
// tokens it still is where the tensor-core kernel's tiles are narrow (few weight rows per SM), and no longer where
// they are 64 rows or taller; beyond two tokens the tensor-core kernel always is.
inline bool gemv_supported(const Params& p) {
  if (p.tokens > 2 || p.d_in % 32 != 0 || gemv_smem_bytes(p.tokens, p.d_in) > 200 * 1024) return false;
  return p.tokens == 1 || infer_pick_tile_n(p.d_out, 1, sm_count()) < 64;
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
  a.nb = a.tile_n / 16;
  a.tiles_n = ceil_div(p.d_out, a.tile_n);
  a.num_kb = ceil_div(p.d_in, INF_BK);
  a.group_shift = -1;
  for (int sh = 5; sh < 31; ++sh)
    if ((1 << sh) == p.group) a.group_shift = sh;
  a.s16 = s16; a.b16 = b16;
  a.one_group = (p.group % INF_BK == 0) ? 1 : 0;
  a.Y = reinterpret_cast<__nv_bfloat16*>(Y);
  CUtensorMap tx, tc;
  a.x_rows = std::min(INF_M, (p.tokens + 7) / 8 * 8);
  if (!make_tmap_bf16(&tx, X, p.tokens, p.d_in, a.x_rows)) return cuda_fail();
  if (!make_tmap_words(&tc, codes, p.d_out, ((uint64_t)p.d_in * p.bits) >> 5, 4 * p.bits, a.tile_n)) return cuda_fail();
  // shared-memory plan: the code ring, then as many operand stages as fit
  a.x_bytes = (uint32_t)a.x_rows * 256u;                        // two boxes of x_rows x 128 bytes
  a.w_bytes = (uint32_t)a.tile_n * 256u;
  a.c_bytes = (uint32_t)(((size_t)a.tile_n * 4 * p.bits * 4 + 127) / 128 * 128);
  // An MMA reads 128 rows of 128 bytes from each X box whatever x_rows is (the extra rows' results are never
  // stored); the code ring and the slack behind the last stage keep those reads inside the allocation.
  const size_t slack = a.x_rows < INF_M ? (size_t)INF_M * 128 : 0;
  const size_t fixed = 1024 + (size_t)INF_C_STAGES * a.c_bytes + sizeof(InferBarriers) + slack;
  a.op_stages = (int)std::min<size_t>(INF_MAX_OP_STAGES, (INF_SMEM_LIMIT - fixed) / (a.x_bytes + a.w_bytes));
  if (a.op_stages < 2) return L4Q_ERR_UNSUPPORTED;
  a.workers = std::min(INF_WORKERS, a.nb * a.op_stages);
  const size_t smem = fixed + (size_t)a.op_stages * (a.x_bytes + a.w_bytes);
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
