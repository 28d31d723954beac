// Initialisation of the quantization parameters (Sec. 3.3, Eq. 15; App. B) for groups of 32, 64 or 128 elements of a
// bf16 weight, fed by TMA: one thread streams 128 x 128 tiles into a ring of six 128-byte-swizzled stages, two sets
// of four warps take the tiles in turn, a thread owning one weight row of the tile (its groups lie inside the row, so
// there is nothing to exchange between threads).  The arithmetic per group is that of k_init_params.
#pragma once

#include "l4q_common.cuh"
#include "l4q_gemm.cuh"
#include "l4q_ptx.cuh"
#include "l4q_quant.cuh"

namespace l4q {

constexpr int IT_ROWS = 128, IT_COLS = 128, IT_STAGES = 6, IT_STAGE_BYTES = IT_ROWS * IT_COLS * 2;
constexpr int IT_SETS = 2;                               // consumer sets of 128 threads
constexpr int IT_THREADS = 32 + IT_SETS * 128;

struct __align__(8) InitBarriers {
  uint64_t full[IT_STAGES], empty[IT_STAGES];
  volatile uint32_t abort;
};

template <int GROUP>
__global__ void __launch_bounds__(IT_THREADS, 1)
k_init_params_tma(const __grid_constant__ CUtensorMap tmap_w, Params p, int method, bool signed_grid,
                  float* __restrict__ s_out, float* __restrict__ b_out, int tiles_m, int tiles_n) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  InitBarriers* bars = reinterpret_cast<InitBarriers*>(smem + (size_t)IT_STAGES * IT_STAGE_BYTES);
  if (threadIdx.x == 0) {
    for (int i = 0; i < IT_STAGES; ++i) { ptx::mbar_init(&bars->full[i], 1); ptx::mbar_init(&bars->empty[i], 128); }
    bars->abort = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tmap_w);
  }
  __syncthreads();
  const int total = tiles_m * tiles_n;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp == 0) {
    if (lane == 0) {                                     // loads: column-panel-major, like the weight-tile kernel
      int stage = 0; uint32_t phase = 0;
      for (int t = blockIdx.x; t < total; t += gridDim.x) {
        if (!bounded_wait(&bars->empty[stage], phase ^ 1, bars)) break;
        const int tn = t / tiles_m, tm = t - tn * tiles_m;
        uint8_t* dst = smem + (size_t)stage * IT_STAGE_BYTES;
        ptx::mbar_arrive_expect_tx(&bars->full[stage], IT_STAGE_BYTES);
        ptx::tma_load_2d(dst, &tmap_w, &bars->full[stage], tn * IT_COLS, tm * IT_ROWS);
        ptx::tma_load_2d(dst + IT_STAGE_BYTES / 2, &tmap_w, &bars->full[stage], tn * IT_COLS + 64, tm * IT_ROWS);
        if (++stage == IT_STAGES) { stage = 0; phase ^= 1; }
      }
    }
  } else {
    // set `set` takes the CTA's tiles set, set + 2, ...: stages set, set + 2, set + 4, then round again
    const int set = (warp - 1) >> 2, row = ((warp - 1) & 3) * 32 + lane;
    const float qn_s = -(float)(1 << (p.bits - 1)), qp_s = (float)((1 << (p.bits - 1)) - 1);
    const float inv_n = 1.f / (float)GROUP, inv_half = 1.f / (float)(1 << (p.bits - 1));
    const uint32_t smem_a = ptx::smem_u32(smem) + (uint32_t)(row * 128);
    const uint32_t sw = (uint32_t)(row & 7);
    int stage = set; uint32_t phase = 0;
    int i = set;
    for (int t = blockIdx.x + set * (int)gridDim.x; t < total; t += IT_SETS * (int)gridDim.x, i += IT_SETS) {
      if (!bounded_wait(&bars->full[stage], phase, bars)) break;
      const int tn = t / tiles_m, tm = t - tn * tiles_m;
      const int o = tm * IT_ROWS + row;
      const uint32_t base = smem_a + (uint32_t)stage * IT_STAGE_BYTES;
      // 16-byte chunk c (8 values) of the row: 64-column half c >> 3, swizzled position (c & 7) ^ (row & 7)
      auto chunk = [&](int c) { return ptx::lds128(base + (uint32_t)(c >> 3) * (IT_STAGE_BYTES / 2) + ((((uint32_t)c & 7u) ^ sw) << 4)); };
#pragma unroll
      for (int j = 0; j < IT_COLS / GROUP; ++j) {
        float lo = INFINITY, hi = -INFINITY, sum = 0.f;
#pragma unroll
        for (int c = 0; c < GROUP / 8; ++c) {
          const uint4 r = chunk(j * (GROUP / 8) + c);
          const float v[8] = {bf16_lo(r.x), bf16_hi(r.x), bf16_lo(r.y), bf16_hi(r.y), bf16_lo(r.z), bf16_hi(r.z), bf16_lo(r.w), bf16_hi(r.w)};
#pragma unroll
          for (int e = 0; e < 8; ++e) { lo = fminf(lo, v[e]); hi = fmaxf(hi, v[e]); sum += v[e]; }
        }
        float sc = 0.f, bs = 0.f;
        if (method == INIT_LSQ_PLUS) {
          const float mu = sum * inv_n;
          float ss = 0.f;                                // second pass over the stage: sum of squared deviations
#pragma unroll
          for (int c = 0; c < GROUP / 8; ++c) {
            const uint4 r = chunk(j * (GROUP / 8) + c);
            const float v[8] = {bf16_lo(r.x), bf16_hi(r.x), bf16_lo(r.y), bf16_hi(r.y), bf16_lo(r.z), bf16_hi(r.z), bf16_lo(r.w), bf16_hi(r.w)};
#pragma unroll
            for (int e = 0; e < 8; ++e) ss = fmaf(v[e] - mu, v[e] - mu, ss);
          }
          const float sigma = sqrtf(ss * inv_n);
          sc = fmaxf(fabsf(mu - 3.f * sigma), fabsf(mu + 3.f * sigma)) * inv_half;
        } else if (method == INIT_SYMM) {
          sc = fmaxf(fabsf(lo), fabsf(hi)) * inv_half;
        } else if (method == INIT_ASYMM) {
          sc = fmaxf((hi - lo) / (qp_s - qn_s), 1e-8f);
          bs = signed_grid ? lo - sc * qn_s : lo;        // unsigned grid: b' = b + s Q_N = min W exactly
        } else {
          sc = fmaxf(fabsf(lo / qn_s), fabsf(hi / qp_s));
        }
        sc = fmaxf(sc, 1e-8f);
        if (!signed_grid && method != INIT_ASYMM) bs = sc * qn_s;   // b = 0 on the signed grid
        const int col = tn * IT_COLS + j * GROUP;
        if (o < p.d_out && col < p.d_in) {
          const size_t at = (size_t)o * p.ngroups + (size_t)(col / GROUP);
          s_out[at] = sc; b_out[at] = bs;
        }
      }
      ptx::mbar_arrive(&bars->empty[stage]);
      stage += IT_SETS;
      if (stage >= IT_STAGES) { stage -= IT_STAGES; phase ^= 1; }
    }
  }
  if (bars->abort) {
    for (int k = 0; k < 64; ++k) __nanosleep(1000);      // let copies in flight land before shared memory is released
  }
  __syncthreads();
}

inline bool init_tma_supported(const Params& p) { return p.group == 32 || p.group == 64 || p.group == 128; }

// W: bf16 [d_out, d_in] row-major.
inline l4q_status launch_init_tma(const Params& p, int method, bool signed_grid, const void* W, float* s, float* b,
                                  cudaStream_t st) {
  CUtensorMap t_w;
  if (!make_tmap_bf16(&t_w, W, p.d_out, p.d_in, IT_ROWS)) return cuda_fail();
  const int tiles_m = ceil_div(p.d_out, IT_ROWS), tiles_n = ceil_div(p.d_in, IT_COLS);
  const size_t smem = 1024 + (size_t)IT_STAGES * IT_STAGE_BYTES + sizeof(InitBarriers);
  const int grid = std::min(tiles_m * tiles_n, sm_count());
  auto launch = [&](auto kern) -> l4q_status {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return cuda_fail();
    kern<<<grid, IT_THREADS, smem, st>>>(t_w, p, method, signed_grid, s, b, tiles_m, tiles_n);
    return cudaGetLastError() == cudaSuccess ? L4Q_OK : L4Q_ERR_CUDA;
  };
  if (p.group == 32) return launch(k_init_params_tma<32>);
  if (p.group == 64) return launch(k_init_params_tma<64>);
  return launch(k_init_params_tma<128>);
}

}  // namespace l4q
