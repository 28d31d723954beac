// Fully quantized inference (Sec. 3.2, App. F): Y = X W_q^T where only the export of l4q_pack_int is
// kept -- bit-packed unsigned codes u and one fp16 scale / offset per group, W_q = u * s16 + b16.
//
// The regime of the paper's deployment measurements is a handful of tokens per step (batch 1..64), so the
// kernel is bound by reading the packed weight once (bits/8 bytes per weight) and is built around that:
//   * tokens are the MMA's M (one 128-row tile, zero-filled beyond the batch), output features its N, in
//     tiles of 64 rows of W so that even a 4096-row layer gives every SM work;
//   * per 128-deep k-block, TMA brings the X tile (128-byte-swizzled) and the tile's packed code words
//     (64 rows x 64 or 48 bytes) into shared memory; 256 dequantizer threads (one per weight row and 32
//     codes) turn the words into bf16 W_q = u * s + b (fp32 arithmetic) and write the MMA's B operand in
//     the swizzled K-major layout; one thread issues tcgen05.mma (bf16 x bf16 -> fp32 in tensor memory);
//   * 4 epilogue warps drain the 128 x 64 accumulator of the previous tile meanwhile.
// Roles (512 threads): warp 0 = TMA, warp 1 = MMA issuer + TMEM owner, warps 4..7 = epilogue,
// warps 8..15 = dequantizers.  Every mbarrier wait is bounded (bounded_wait).
#pragma once

#include "l4q_common.cuh"
#include "l4q_gemm.cuh"
#include "l4q_ptx.cuh"
#include "l4q_wtile.cuh"

namespace l4q {

constexpr int INF_M = 128;                 // tokens per tile (MMA M)
constexpr int INF_N = 64;                  // weight rows per tile (MMA N)
constexpr int INF_BK = 128;                // k per pipeline stage
constexpr int INF_STAGES = 4;
constexpr int INF_THREADS = 512;
constexpr int INF_DEQ_THREADS = 256;       // warps 8..15
constexpr int INF_X_BYTES = INF_M * INF_BK * 2;      // 32 KB: two 128 x 64 swizzled boxes
constexpr int INF_W_BYTES = INF_N * INF_BK * 2;      // 16 KB: two 64 x 64 swizzled tiles
constexpr int INF_C_BYTES = 4096;                    // packed codes of the stage: 64 rows x (16 | 12) words
constexpr int INF_STAGE_BYTES = INF_X_BYTES + INF_W_BYTES + INF_C_BYTES;
constexpr int INF_ACC = 2;

struct InferArgs {
  int tokens, d_in, d_out, bits, group, ngroups;
  int tiles_m, tiles_n, num_kb;
  const __half *s16, *b16;
  __nv_bfloat16* Y;
};

struct __align__(8) InferBarriers {
  uint64_t full_in[INF_STAGES];            // X tile and code words have landed
  uint64_t full_w[INF_STAGES];             // the dequantized B operand of the stage is complete
  uint64_t empty[INF_STAGES];              // the MMAs reading the stage have completed
  uint64_t tmem_full[INF_ACC], tmem_empty[INF_ACC];
  uint32_t tmem_base;
  volatile uint32_t abort;
};

inline size_t infer_smem_bytes() { return 1024 + (size_t)INF_STAGES * INF_STAGE_BYTES + sizeof(InferBarriers); }

// 32 unsigned codes of one weight row, starting at a multiple of 32 codes, from the LSB-first bitstream.
template <int BITS>
__device__ __forceinline__ void unpack_codes32(const uint32_t (&w)[BITS], float (&u)[32]) {
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const int bit = j * BITS, wd = bit >> 5, off = bit & 31;
    uint32_t v = w[wd] >> off;
    if (off + BITS > 32) v |= w[wd + 1] << (32 - off);
    // integer -> float without the conversion pipe: 2^23 + v has v in its low mantissa bits
    u[j] = __uint_as_float(0x4B000000u | (v & ((1u << BITS) - 1u))) - 8388608.0f;
  }
}

template <int BITS>
__global__ void __launch_bounds__(INF_THREADS, 1)
k_infer_bf16(const __grid_constant__ CUtensorMap tmap_x,      // X [tokens, d_in] bf16, box 64 x 128, swizzled
             const __grid_constant__ CUtensorMap tmap_c,      // codes [d_out, words] uint32, box (4 BITS) x 64
             const InferArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  InferBarriers* bars = reinterpret_cast<InferBarriers*>(smem + (size_t)INF_STAGES * INF_STAGE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = a.tiles_m * a.tiles_n;
  constexpr int CW = 4 * BITS;                                 // code words per row and stage (128 codes)
  auto x_tile = [&](int st) { return smem + (size_t)st * INF_STAGE_BYTES; };
  auto w_tile = [&](int st) { return smem + (size_t)st * INF_STAGE_BYTES + INF_X_BYTES; };
  auto c_tile = [&](int st) { return smem + (size_t)st * INF_STAGE_BYTES + INF_X_BYTES + INF_W_BYTES; };

  if (threadIdx.x == 0) {
    for (int i = 0; i < INF_STAGES; ++i) {
      ptx::mbar_init(&bars->full_in[i], 1);
      ptx::mbar_init(&bars->full_w[i], INF_DEQ_THREADS);
      ptx::mbar_init(&bars->empty[i], 1);
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
    ptx::tmem_alloc(&bars->tmem_base, INF_ACC * INF_N);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;

  if (warp == 0) {
    // ------------------------------ TMA: X tile and code words ------------------------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      for (int t = blockIdx.x; t < num_tiles && !bars->abort; t += gridDim.x) {
        const int m0 = (t / a.tiles_n) * INF_M, n0 = (t % a.tiles_n) * INF_N;
        for (int kb = 0; kb < a.num_kb && !bars->abort; ++kb) {
          bounded_wait(&bars->empty[stage], phase ^ 1, bars);
          if (bars->abort) break;
          ptx::mbar_arrive_expect_tx(&bars->full_in[stage], INF_X_BYTES + INF_N * CW * 4);
          ptx::tma_load_2d(x_tile(stage), &tmap_x, &bars->full_in[stage], kb * INF_BK, m0);
          ptx::tma_load_2d(x_tile(stage) + INF_X_BYTES / 2, &tmap_x, &bars->full_in[stage], kb * INF_BK + 64, m0);
          ptx::tma_load_2d(c_tile(stage), &tmap_c, &bars->full_in[stage], kb * CW, n0);
          if (++stage == INF_STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(INF_M, INF_N, false, false);
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      for (int t = blockIdx.x; t < num_tiles && !bars->abort; t += gridDim.x) {
        bounded_wait(&bars->tmem_empty[acc], acc_phase ^ 1, bars);
        if (bars->abort) break;
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * INF_N);
        for (int kb = 0; kb < a.num_kb; ++kb) {
          bounded_wait(&bars->full_in[stage], phase, bars);
          bounded_wait(&bars->full_w[stage], phase, bars);
          if (bars->abort) break;
          ptx::tc_fence_after_sync();
          const uint32_t xa = ptx::smem_u32(x_tile(stage)), wa = ptx::smem_u32(w_tile(stage));
#pragma unroll
          for (int ks = 0; ks < INF_BK / UMMA_K; ++ks) {     // 8 steps of 16; steps 4..7 are the second 64-wide tile
            const uint64_t da = ptx::make_smem_desc_sw128(xa + (ks >> 2) * (INF_X_BYTES / 2) + (ks & 3) * 32, 16, 1024);
            const uint64_t db = ptx::make_smem_desc_sw128(wa + (ks >> 2) * (INF_W_BYTES / 2) + (ks & 3) * 32, 16, 1024);
            ptx::mma_bf16_ss(d_tmem, da, db, idesc, (kb | ks) != 0 ? 1u : 0u);
          }
          ptx::mma_commit(&bars->empty[stage]);
          if (++stage == INF_STAGES) { stage = 0; phase ^= 1; }
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
      const int m0 = (t / a.tiles_n) * INF_M, n0 = (t % a.tiles_n) * INF_N;
      bounded_wait(&bars->tmem_full[acc], acc_phase, bars);
      ptx::tc_fence_after_sync();
      const int tok = m0 + quarter * 32 + lane;
#pragma unroll
      for (int c = 0; c < INF_N / 32; ++c) {
        uint32_t raw[32];
        ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * INF_N + c * 32), raw);
        ptx::tmem_ld_wait();
        if (c == INF_N / 32 - 1) {
          ptx::tc_fence_before_sync();
          ptx::mbar_arrive(&bars->tmem_empty[acc]);
        }
        if (tok < a.tokens) {
          __nv_bfloat16* dst = a.Y + (size_t)tok * a.d_out + n0 + c * 32;
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            if (n0 + c * 32 + v * 8 < a.d_out) {
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
    const int pt = threadIdx.x - 256;                          // 0 .. 255
    const int row = pt >> 2, q = pt & 3;                       // row of the tile, 32-code quarter of the k-block
    int stage = 0; uint32_t phase = 0;
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
      const int n0 = (t % a.tiles_n) * INF_N;
      const int o = n0 + row;
      const bool row_ok = o < a.d_out;
      // s, b of the group of this thread's 32 codes (group size is a multiple of 32), fetched one k-block ahead
      auto load_sb = [&](int kb, float& s_, float& b_) {
        const int k = kb * INF_BK + q * 32;
        if (row_ok && k < a.d_in) {
          const size_t gi = (size_t)o * a.ngroups + k / a.group;
          s_ = __half2float(__ldg(a.s16 + gi));
          b_ = __half2float(__ldg(a.b16 + gi));
        } else {
          s_ = 0.f; b_ = 0.f;                                  // rows / columns beyond the weight contribute nothing
        }
      };
      float s_next, b_next;
      load_sb(0, s_next, b_next);
      for (int kb = 0; kb < a.num_kb; ++kb) {
        const float s_ = s_next, b_ = b_next;
        if (kb + 1 < a.num_kb) load_sb(kb + 1, s_next, b_next);
        bounded_wait(&bars->full_in[stage], phase, bars);      // the code words have landed
        const uint8_t* crow = c_tile(stage) + row * (CW * 4) + q * (BITS * 4);
        uint32_t w[BITS];
        if constexpr (BITS == 4) {
          const uint4 v = *reinterpret_cast<const uint4*>(crow);
          w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
        } else {
#pragma unroll
          for (int i = 0; i < BITS; ++i) w[i] = reinterpret_cast<const uint32_t*>(crow)[i];
        }
        float u[32];
        unpack_codes32<BITS>(w, u);
        // W_q = u * s + b (Eq. 9 on the unsigned code), bf16, into the K-major swizzled B operand:
        // 64-k tile q >> 1, 16-byte chunks (q & 1) * 4 .. + 3 of row `row`
        uint8_t* wrow = w_tile(stage) + (q >> 1) * (INF_W_BYTES / 2) + row * 128;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint4 o4;
          o4.x = pack_bf16x2(fmaf(u[c * 8 + 0], s_, b_), fmaf(u[c * 8 + 1], s_, b_));
          o4.y = pack_bf16x2(fmaf(u[c * 8 + 2], s_, b_), fmaf(u[c * 8 + 3], s_, b_));
          o4.z = pack_bf16x2(fmaf(u[c * 8 + 4], s_, b_), fmaf(u[c * 8 + 5], s_, b_));
          o4.w = pack_bf16x2(fmaf(u[c * 8 + 6], s_, b_), fmaf(u[c * 8 + 7], s_, b_));
          *reinterpret_cast<uint4*>(wrow + ((((q & 1) * 4 + c) ^ (row & 7)) << 4)) = o4;
        }
        ptx::fence_proxy_async_smem();                         // the operand is read by the tensor cores
        ptx::mbar_arrive(&bars->full_w[stage]);
        if (++stage == INF_STAGES) { stage = 0; phase ^= 1; }
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
    ptx::tmem_dealloc(tmem_base, INF_ACC * INF_N);
  }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------

inline bool infer_supported(const Params& p) {
  if (p.bits != 3 && p.bits != 4) return false;
  if (p.group % 32 != 0) return false;                          // a thread's 32 codes share one group
  const long long bits_per_row = (long long)p.d_in * p.bits;
  if (bits_per_row % 32 != 0 || ((bits_per_row / 32) * 4) % 16 != 0) return false;   // TMA row pitch of the codes
  return true;
}

inline l4q_status launch_infer_bf16(const Params& p, const void* X, const uint32_t* codes, const __half* s16,
                                    const __half* b16, void* Y, cudaStream_t st) {
  InferArgs a{};
  a.tokens = p.tokens; a.d_in = p.d_in; a.d_out = p.d_out; a.bits = p.bits; a.group = p.group; a.ngroups = p.ngroups;
  a.tiles_m = ceil_div(p.tokens, INF_M);
  a.tiles_n = ceil_div(p.d_out, INF_N);
  a.num_kb = ceil_div(p.d_in, INF_BK);
  a.s16 = s16; a.b16 = b16;
  a.Y = reinterpret_cast<__nv_bfloat16*>(Y);
  CUtensorMap tx, tc;
  if (!make_tmap_bf16(&tx, X, p.tokens, p.d_in, INF_M)) return L4Q_ERR_CUDA;
  if (!make_tmap_words(&tc, codes, p.d_out, ((uint64_t)p.d_in * p.bits) >> 5, 4 * p.bits, INF_N)) return L4Q_ERR_CUDA;
  const size_t smem = infer_smem_bytes();
  const int grid = std::min(a.tiles_m * a.tiles_n, sm_count());
  auto launch = [&](auto kern) -> l4q_status {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return L4Q_ERR_CUDA;
    kern<<<grid, INF_THREADS, smem, st>>>(tx, tc, a);
    return cudaGetLastError() == cudaSuccess ? L4Q_OK : L4Q_ERR_CUDA;
  };
  return p.bits == 4 ? launch(k_infer_bf16<4>) : launch(k_infer_bf16<3>);
}

}  // namespace l4q
