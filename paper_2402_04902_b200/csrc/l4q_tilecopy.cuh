// Measurement helper: what the memory system gives a kernel with the weight-tile kernel's traffic and nothing
// else to do.  Persistent CTAs (one per SM) move a bf16 matrix in 128 x 128 tiles -- TMA loads into a ring of
// 128-byte-swizzled stages and, in copy mode, TMA stores of the same stages -- with one loading and one
// storing thread per CTA and no arithmetic at all.  Its time is the floor of any kernel that reads a weight
// once (read mode: the export) or reads and rewrites it (copy mode: the dequantize step), launch and ramp
// included, on the size of one layer rather than on the gigabytes a bandwidth peak is quoted on.
#pragma once

#include "l4q_common.cuh"
#include "l4q_gemm.cuh"
#include "l4q_ptx.cuh"

namespace l4q {

constexpr int TC_ROWS = 128, TC_COLS = 128, TC_STAGES = 6, TC_STAGE_BYTES = TC_ROWS * TC_COLS * 2;

struct __align__(8) TileCopyBarriers {
  uint64_t full[TC_STAGES], empty[TC_STAGES];
  volatile uint32_t abort;
};

__global__ void __launch_bounds__(64, 1)
k_tile_copy(const __grid_constant__ CUtensorMap tmap_in, const __grid_constant__ CUtensorMap tmap_out, int tiles_m,
            int tiles_n, int cols, int do_store) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  TileCopyBarriers* bars = reinterpret_cast<TileCopyBarriers*>(smem + (size_t)TC_STAGES * TC_STAGE_BYTES);
  if (threadIdx.x == 0) {
    for (int i = 0; i < TC_STAGES; ++i) { ptx::mbar_init(&bars->full[i], 1); ptx::mbar_init(&bars->empty[i], 1); }
    bars->abort = 0;
    ptx::fence_mbar_init();
  }
  __syncthreads();
  const int total = tiles_m * tiles_n;
  if (threadIdx.x == 0) {                              // loads: column-panel-major, like the weight-tile kernel
    int stage = 0; uint32_t phase = 0;
    for (int t = blockIdx.x; t < total; t += gridDim.x) {
      if (!bounded_wait(&bars->empty[stage], phase ^ 1, bars)) break;
      const int tn = t / tiles_m, tm = t - tn * tiles_m;
      uint8_t* dst = smem + (size_t)stage * TC_STAGE_BYTES;
      ptx::mbar_arrive_expect_tx(&bars->full[stage], TC_STAGE_BYTES);
      ptx::tma_load_2d(dst, &tmap_in, &bars->full[stage], tn * TC_COLS, tm * TC_ROWS);
      ptx::tma_load_2d(dst + TC_STAGE_BYTES / 2, &tmap_in, &bars->full[stage], tn * TC_COLS + 64, tm * TC_ROWS);
      if (++stage == TC_STAGES) { stage = 0; phase ^= 1; }
    }
  } else if (threadIdx.x == 32) {                      // stores (or nothing), then the stage goes back
    int stage = 0; uint32_t phase = 0;
    for (int t = blockIdx.x; t < total; t += gridDim.x) {
      if (!bounded_wait(&bars->full[stage], phase, bars)) break;
      if (do_store) {
        const int tn = t / tiles_m, tm = t - tn * tiles_m;
        const uint8_t* src = smem + (size_t)stage * TC_STAGE_BYTES;
        ptx::tma_store_2d(&tmap_out, src, tn * TC_COLS, tm * TC_ROWS);
        if (tn * TC_COLS + 64 < cols) ptx::tma_store_2d(&tmap_out, src + TC_STAGE_BYTES / 2, tn * TC_COLS + 64, tm * TC_ROWS);
        ptx::bulk_commit_group();
        ptx::bulk_wait_group_read0();
      }
      ptx::mbar_arrive(&bars->empty[stage]);
      if (++stage == TC_STAGES) { stage = 0; phase ^= 1; }
    }
    if (do_store) ptx::bulk_wait_group0();
  }
  if (bars->abort) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);    // let copies in flight land before shared memory is released
  }
  __syncthreads();
}

// src, dst: bf16 [rows, cols] row-major (cols a multiple of 8, pointers 16-byte aligned); dst null = read only.
inline l4q_status launch_tile_copy(const void* src, void* dst, int rows, int cols, cudaStream_t st) {
  CUtensorMap t_in, t_out;
  if (!make_tmap_bf16(&t_in, src, rows, cols, TC_ROWS)) return cuda_fail();
  t_out = t_in;
  if (dst && !make_tmap_bf16(&t_out, dst, rows, cols, TC_ROWS)) return cuda_fail();
  const int tiles_m = ceil_div(rows, TC_ROWS), tiles_n = ceil_div(cols, TC_COLS);
  const size_t smem = 1024 + (size_t)TC_STAGES * TC_STAGE_BYTES + sizeof(TileCopyBarriers);
  if (cudaFuncSetAttribute(k_tile_copy, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    cudaGetLastError();
    return cuda_fail();
  }
  k_tile_copy<<<std::min(tiles_m * tiles_n, sm_count()), 64, smem, st>>>(t_in, t_out, tiles_m, tiles_n, cols, dst != nullptr);
  return cudaGetLastError() == cudaSuccess ? L4Q_OK : L4Q_ERR_CUDA;
}

}  // namespace l4q
