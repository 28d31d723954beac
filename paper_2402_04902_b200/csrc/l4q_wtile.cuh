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
//   * 16 epilogue warps in two groups of eight; a group owns every second tile of the CTA and two of the four
//     accumulator stages, a thread one weight row and one 64-column half of the group's tile.  It reads the
//     merge from tensor memory with tcgen05.ld, the W0 tile from shared memory in 16-byte pieces, and does
//     the quantizer arithmetic.  The groups meet only through mbarriers, so two tiles are worked on per SM
//     while the loads, merges and stores of their neighbours are in flight;
//   * nothing but that arithmetic is left to the epilogue warps where the caller provides scratch: the MMA
//     operands of the merge (the tile's slices of A and B, each value split into tf32 head / tail, K-major
//     with the 128-byte swizzle) are written once per launch for every row and column panel by
//     k_split_operands, laid out as they stand in shared memory, and come in by two bulk copies per tile;
//     s and b of the tile's rows come in by TMA with the W0 tile (where their row pitch allows).
//
// Roles (640 threads): warp 0 = TMA loads (W0, s, b), warp 1 = MMA issuer + TMEM owner, warp 2 = TMA stores,
// warp 3 = bulk copies of the operand images (one thread each), warps 4..19 = epilogue (warp w: TMEM lane
// quarter w % 4, group (w - 4) / 8, column half ((w - 4) / 4) % 2).  Without operand images a group builds
// the operands of its next tile itself once the MMAs that last read the operand buffer have completed (two
// buffers up to rank 32, one at rank 64); without TMA boxes of s and b it copies those of its next tile's rows
// to scratch in shared memory and meets at a named barrier per tile.
// Every mbarrier wait is bounded (see bounded_wait); there is no block-level barrier after set-up.
#pragma once

#include "l4q_common.cuh"
#include "l4q_gemm.cuh"
#include "l4q_ptx.cuh"

namespace l4q {

constexpr int WT2_ROWS = 128, WT2_COLS = 128;
constexpr int WT2_THREADS = 640;
constexpr int WT2_FIRST_EPI_WARP = 4;
constexpr int WT2_EPI_THREADS = 512;
constexpr int WT2_GROUPS = 2;                       // epilogue warp groups; each owns every second tile of the CTA
constexpr int WT2_GROUP_THREADS = WT2_EPI_THREADS / WT2_GROUPS;
constexpr int WT2_ACC = 4;                          // accumulator stages of 128 TMEM columns
constexpr int WT2_STAGE_BYTES = WT2_ROWS * WT2_COLS * 2;   // one bf16 tile: two 128 x 64 swizzled boxes
constexpr int WT2_ATOM_BYTES = 128 * 128;           // 128 rows x 32 tf32 (one 128-byte swizzle atom along K)
constexpr int WT2_MAX_STAGES = 4;

enum { WT2_DEQUANT = 0, WT2_DEQUANT_F = 1, WT2_PACK = 2 };

struct WtileArgs {
  Params p;
  const float *A, *B, *s, *b;
  __half *s16, *b16;       // WT2_PACK
  __half* F;               // WT2_DEQUANT_F: the factor array (factor_index layout)
  const uint8_t* op_img;   // optional: the split MMA operands of every panel, ready made (see k_split_operands)
  int tiles_m, tiles_n;
  int n_stages;            // W0 stages in shared memory (2..4)
  int n_out;               // staging buffers for the second output (F or codes): 0, 1 or 2
  int out_bytes;           // bytes of one such buffer
  int atoms;               // swizzle atoms per operand row: ceil(2 rank / 32)
  int ngt;                 // upper bound of the quantization groups a 128-column tile intersects
  int n_opbuf;             // MMA operand buffers ([A slice | B slice] each): 1 or 2
  int group_shift;         // log2(group size) if it is a power of two, else -1
  int sb_box;              // groups per row of the s / b boxes that TMA brings in with the W0 tile; 0: the epilogue
                           // warps stage s and b themselves
};

// column / group size without a division in the common power-of-two case
__device__ __forceinline__ int group_of(const WtileArgs& a, int col) {
  return a.group_shift >= 0 ? (col >> a.group_shift) : (col / a.p.group);
}

struct __align__(8) WtileBarriers {
  uint64_t full[WT2_MAX_STAGES];      // W0 tile has landed in the stage
  uint64_t empty[WT2_MAX_STAGES];     // the stage may be overwritten (its store has read it)
  uint64_t written[WT2_MAX_STAGES];   // the epilogue has written the stage's outputs
  uint64_t out_empty[2];              // second-output staging buffer may be overwritten
  uint64_t prep_full[2];              // split LoRA operands are complete in operand buffer b
  uint64_t tmem_full[WT2_ACC], tmem_empty[WT2_ACC];
  uint32_t tmem_base;
  volatile uint32_t abort;
};

// s and b in shared memory: per epilogue thread [s x ngt | b x ngt] floats of its weight row (1 KB multiples
// in total); a thread reads and writes its own entry only.
__host__ __device__ inline size_t wtile_sb_bytes(int ngt) { return (size_t)WT2_EPI_THREADS * 2 * ngt * sizeof(float); }

// With sb_box: per W0 stage one box [128 rows][sb_box] of s and one of b.
__host__ __device__ inline size_t wtile_sb_region_bytes(const WtileArgs& a) {
  return a.sb_box ? (size_t)a.n_stages * 2 * WT2_ROWS * a.sb_box * sizeof(float) : wtile_sb_bytes(a.ngt);
}
inline size_t wtile_smem_bytes(const WtileArgs& a) {
  return 1024 + (size_t)a.n_stages * WT2_STAGE_BYTES + (size_t)a.n_out * a.out_bytes +
         2 * (size_t)a.n_opbuf * a.atoms * WT2_ATOM_BYTES + wtile_sb_region_bytes(a) + sizeof(WtileBarriers);
}

// The tiles of one CTA: tile t of the column-panel-major sequence (row tiles of one column panel are
// consecutive) goes to CTA t mod gridDim.x.  Coordinates advance without divisions.
struct TileCursor {
  int t, total, tm, tn, tiles_m, dm, dn;
  int step;
  // the CTA's tiles number first, first + stride, ... of its own sequence
  __device__ explicit TileCursor(const WtileArgs& a, int first = 0, int stride = 1) {
    total = a.tiles_m * a.tiles_n;
    tiles_m = a.tiles_m;
    t = blockIdx.x + first * (int)gridDim.x;
    tn = t / tiles_m; tm = t - tn * tiles_m;
    step = stride * (int)gridDim.x;
    dn = step / tiles_m; dm = step - dn * tiles_m;
  }
  __device__ bool valid() const { return t < total; }
  __device__ void next() {
    t += step; tn += dn; tm += dm;
    if (tm >= tiles_m) { tm -= tiles_m; ++tn; }
  }
  __device__ int m0() const { return tm * WT2_ROWS; }
  __device__ int n0() const { return tn * WT2_COLS; }
  // coordinates of this CTA's tile k (small) steps ahead; false beyond the end
  __device__ bool peek(int k, int& m0_, int& n0_) const {
    if (t + k * step >= total) return false;
    int m = tm + k * dm, n = tn + k * dn;
    while (m >= tiles_m) { m -= tiles_m; ++n; }
    m0_ = m * WT2_ROWS; n0_ = n * WT2_COLS;
    return true;
  }
};

// x = hi + lo with hi, lo representable in tf32 (low 13 mantissa bits clear): hi keeps the leading 10
// mantissa bits of x (truncation), lo the leading bits of the exact remainder.  Plain logic ops.
__device__ __forceinline__ void split_tf32(float x, float& hi, float& lo) {
  hi = __uint_as_float(__float_as_uint(x) & 0xFFFFE000u);
  lo = __uint_as_float(__float_as_uint(x - hi) & 0xFFFFE000u);
}

// MMA operands of one tile in shared memory, K-major with the 128-byte swizzle:
//   acat row n = column n0 + n of the weight:  [ hi(A[0..r, col]) | lo(A[0..r, col]) ]
//   bcat row m = row m0 + m of the weight:      [ hi(B[row, 0..r]) | lo(B[row, 0..r]) ]
// A work item (32 r per tile) is 4 consecutive ranks of one row of each slice.  Item idx takes column
// idx % 128, ranks 4 (idx / 128) of the A slice -- a warp reads 32 consecutive columns of one rank, coalesced --
// and the idx-th 16 bytes of the B slice, which is one contiguous block of 128 r floats, so a warp reads 512
// consecutive bytes.
struct OperandItem { float av[4]; float4 bv; };

__device__ __forceinline__ void operand_a_load(const WtileArgs& a, int n0, int idx, float (&av)[4]) {
  const Params& p = a.p;
  const int row = idx & 127, kc = idx >> 7, col = n0 + row;
#pragma unroll
  for (int e = 0; e < 4; ++e) av[e] = (col < p.d_in) ? __ldg(a.A + (size_t)(4 * kc + e) * p.d_in + col) : 0.f;
}

__device__ __forceinline__ void operand_b_load(const WtileArgs& a, int m0, int idx, float4& bv) {
  const Params& p = a.p;
  const int rq = p.rank >> 2;                        // 16-byte pieces per row of B
  const int brow = idx / rq;
  bv = (m0 + brow < p.d_out) ? __ldg(reinterpret_cast<const float4*>(a.B + (size_t)m0 * p.rank) + idx)
                             : make_float4(0.f, 0.f, 0.f, 0.f);
}

__device__ __forceinline__ void operand_a_store(const WtileArgs& a, int idx, const float (&av)[4], uint8_t* acat) {
  const int row = idx & 127, kc = idx >> 7;
  float ah[4], al[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) split_tf32(av[e], ah[e], al[e]);
  const int ch = kc, cl = (a.p.rank >> 2) + kc;      // 16-byte chunk index of the head / tail within the row
  const uint32_t off_h = (uint32_t)(ch >> 3) * WT2_ATOM_BYTES + row * 128 + (((ch & 7) ^ (row & 7)) << 4);
  const uint32_t off_l = (uint32_t)(cl >> 3) * WT2_ATOM_BYTES + row * 128 + (((cl & 7) ^ (row & 7)) << 4);
  *reinterpret_cast<float4*>(acat + off_h) = make_float4(ah[0], ah[1], ah[2], ah[3]);
  *reinterpret_cast<float4*>(acat + off_l) = make_float4(al[0], al[1], al[2], al[3]);
}

__device__ __forceinline__ void operand_b_store(const WtileArgs& a, int idx, const float4& bv, uint8_t* bcat) {
  const int rq = a.p.rank >> 2;
  const int brow = idx / rq, bkc = idx - brow * rq;
  const float bvv[4] = {bv.x, bv.y, bv.z, bv.w};
  float bh[4], bl[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) split_tf32(bvv[e], bh[e], bl[e]);
  const int bch = bkc, bcl = rq + bkc;
  const uint32_t boff_h = (uint32_t)(bch >> 3) * WT2_ATOM_BYTES + brow * 128 + (((bch & 7) ^ (brow & 7)) << 4);
  const uint32_t boff_l = (uint32_t)(bcl >> 3) * WT2_ATOM_BYTES + brow * 128 + (((bcl & 7) ^ (brow & 7)) << 4);
  *reinterpret_cast<float4*>(bcat + boff_h) = make_float4(bh[0], bh[1], bh[2], bh[3]);
  *reinterpret_cast<float4*>(bcat + boff_l) = make_float4(bl[0], bl[1], bl[2], bl[3]);
}

__device__ __forceinline__ void operand_item_load(const WtileArgs& a, int m0, int n0, int idx, OperandItem& it) {
  operand_a_load(a, n0, idx, it.av);
  operand_b_load(a, m0, idx, it.bv);
}

__device__ __forceinline__ void operand_item_store(const WtileArgs& a, int idx, const OperandItem& it, uint8_t* acat,
                                                   uint8_t* bcat) {
  operand_a_store(a, idx, it.av, acat);
  operand_b_store(a, idx, it.bv, bcat);
}

// The operand images of all panels, written once per launch of the weight-tile kernel so that its epilogue warps
// need not build them tile by tile: image tn (tn < tiles_n) is the acat block of column panel tn, image
// tiles_n + tm the bcat block of row panel tm, each exactly as it stands in shared memory (op_half bytes), so
// that one bulk copy brings it in.  One block per panel.
// Output buffers of the caller that must start from zero (they are accumulated into with atomics later on the
// stream): cleared by the same launch, which saves one memset launch per buffer.
struct ZeroList { float* ptr[4]; size_t n[4]; };

__global__ void __launch_bounds__(256) k_split_operands(const WtileArgs a, uint8_t* __restrict__ img, const ZeroList zl) {
  {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
#pragma unroll
    for (int b = 0; b < 4; ++b)
      for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < zl.n[b]; e += stride) zl.ptr[b][e] = 0.f;
  }
  const uint32_t op_half = (uint32_t)a.atoms * WT2_ATOM_BYTES;
  const int panel = blockIdx.x;
  uint8_t* dst = img + (size_t)panel * op_half;
  const int n_items = 32 * a.p.rank;
  // chunks of an atom row beyond 2 rank values are never read by the MMAs; the image leaves them as they are
  if (panel < a.tiles_n) {
    for (int idx = threadIdx.x; idx < n_items; idx += blockDim.x) {
      float av[4];
      operand_a_load(a, panel * WT2_COLS, idx, av);
      operand_a_store(a, idx, av, dst);
    }
  } else {
    for (int idx = threadIdx.x; idx < n_items; idx += blockDim.x) {
      float4 bv;
      operand_b_load(a, (panel - a.tiles_n) * WT2_ROWS, idx, bv);
      operand_b_store(a, idx, bv, dst);
    }
  }
}

// Adding and subtracting 1.5 * 2^23 rounds |x| < 2^22 to the nearest integer, ties to even, exactly like
// rintf, on the FP32 add pipe; the low mantissa bits of the intermediate sum hold that integer.
constexpr float kRoundMagic = 12582912.0f;
constexpr int kRoundMagicBits = 0x4B400000;

template <int MODE>
__global__ void __launch_bounds__(WT2_THREADS, 1)
k_wtile_tc(const __grid_constant__ CUtensorMap tmap_w0,     // load:  W0 [d_out, d_in] bf16, box 64 x 128, swizzled
           const __grid_constant__ CUtensorMap tmap_out0,   // store: W_q (same geometry) | codes (uint32 words)
           const __grid_constant__ CUtensorMap tmap_out1,   // store: STE factors (same geometry as W0) | unused
           const __grid_constant__ CUtensorMap tmap_s,      // load:  s [d_out, ngroups] fp32, box sb_box x 128 (if sb_box)
           const __grid_constant__ CUtensorMap tmap_b,      // load:  b, likewise
           const WtileArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* stage_base = smem;
  uint8_t* out_base = stage_base + (size_t)a.n_stages * WT2_STAGE_BYTES;
  uint8_t* op_base = out_base + (size_t)a.n_out * a.out_bytes;          // operand buffer b: [acat | bcat]
  const uint32_t op_half = (uint32_t)a.atoms * WT2_ATOM_BYTES;           // bytes of one acat or bcat
  float* sb_base = reinterpret_cast<float*>(op_base + (size_t)a.n_opbuf * 2 * op_half);
  WtileBarriers* bars = reinterpret_cast<WtileBarriers*>(reinterpret_cast<uint8_t*>(sb_base) + wtile_sb_region_bytes(a));
  const Params& p = a.p;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr bool HAS_OUT1 = (MODE != WT2_DEQUANT);

  if (threadIdx.x == 0) {
    for (int i = 0; i < WT2_MAX_STAGES; ++i) {
      ptx::mbar_init(&bars->full[i], 1);
      ptx::mbar_init(&bars->empty[i], 1);
      ptx::mbar_init(&bars->written[i], WT2_GROUP_THREADS);
    }
    for (int i = 0; i < 2; ++i) ptx::mbar_init(&bars->out_empty[i], 1);
    for (int i = 0; i < 2; ++i) ptx::mbar_init(&bars->prep_full[i], a.op_img ? 1 : WT2_GROUP_THREADS);
    for (int i = 0; i < WT2_ACC; ++i) {
      ptx::mbar_init(&bars->tmem_full[i], 1);
      ptx::mbar_init(&bars->tmem_empty[i], WT2_GROUP_THREADS);
    }
    bars->abort = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tmap_w0);
    ptx::prefetch_tmap(&tmap_out0);
    if (MODE == WT2_DEQUANT_F) ptx::prefetch_tmap(&tmap_out1);
    if (a.sb_box) { ptx::prefetch_tmap(&tmap_s); ptx::prefetch_tmap(&tmap_b); }
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
      for (TileCursor cur(a); !bars->abort && cur.valid(); cur.next()) {
        const int m0 = cur.m0(), n0 = cur.n0();
        bounded_wait(&bars->empty[stage], phase ^ 1, bars);
        if (bars->abort) break;
        uint8_t* dst = stage_base + (size_t)stage * WT2_STAGE_BYTES;
        const uint32_t sb_box_bytes = (uint32_t)(WT2_ROWS * a.sb_box * sizeof(float));
        ptx::mbar_arrive_expect_tx(&bars->full[stage], WT2_STAGE_BYTES + 2 * sb_box_bytes);
        ptx::tma_load_2d(dst, &tmap_w0, &bars->full[stage], n0, m0);
        ptx::tma_load_2d(dst + WT2_STAGE_BYTES / 2, &tmap_w0, &bars->full[stage], n0 + 64, m0);
        if (a.sb_box) {
          // s and b of the tile's rows, from the group column rounded down to a 16-byte boundary
          uint8_t* sdst = reinterpret_cast<uint8_t*>(sb_base) + (size_t)stage * 2 * sb_box_bytes;
          const int x0 = group_of(a, n0) & ~3;
          ptx::tma_load_2d(sdst, &tmap_s, &bars->full[stage], x0, m0);
          ptx::tma_load_2d(sdst + sb_box_bytes, &tmap_b, &bars->full[stage], x0, m0);
        }
        if (++stage == a.n_stages) { stage = 0; phase ^= 1; }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------ merge MMAs --------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_tf32(WT2_ROWS, WT2_COLS);
      const int r = p.rank, ksteps = r >> 3;
      int acc = 0; uint32_t acc_phase = 0;
      int buf = 0; uint32_t buf_phase = 0;
      for (TileCursor cur(a); !bars->abort && cur.valid(); cur.next()) {
        const uint32_t acat_a = ptx::smem_u32(op_base) + (uint32_t)buf * 2 * op_half, bcat_a = acat_a + op_half;
        bounded_wait(&bars->prep_full[buf], buf_phase, bars);
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
        if (++buf == a.n_opbuf) { buf = 0; buf_phase ^= 1; }
      }
    }
    __syncwarp();
  } else if (warp == 2) {
    // ------------------------------ TMA stores --------------------------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      int ob = 0;
      for (TileCursor cur(a); !bars->abort && cur.valid(); cur.next()) {
        const int m0 = cur.m0(), n0 = cur.n0();
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
          // the staging buffer is the tile's block of the factor array as it stands: one contiguous copy
          ptx::bulk_store(a.F + ((size_t)cur.tm * a.tiles_n + cur.tn) * FACTOR_TILE_ELEMS, src1, WT2_STAGE_BYTES);
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
  } else if (warp == 3) {
    // ------------------------------ MMA operands from the ready-made images ----
    if (lane == 0 && a.op_img) {
      const int L = a.n_opbuf;
      int j = 0;
      for (TileCursor cur(a); !bars->abort && cur.valid(); cur.next(), ++j) {
        const int buf = j & (L - 1);
        if (j >= L) {      // the MMAs of tile j - L, the last readers of this buffer, have completed
          bounded_wait(&bars->tmem_full[(j - L) & 3], (uint32_t)(((j - L) >> 2) & 1), bars);
          if (bars->abort) break;
        }
        uint8_t* acat = op_base + (size_t)buf * 2 * op_half;
        ptx::mbar_arrive_expect_tx(&bars->prep_full[buf], 2 * op_half);
        ptx::bulk_load(acat, a.op_img + (size_t)cur.tn * op_half, op_half, &bars->prep_full[buf]);
        ptx::bulk_load(acat + op_half, a.op_img + (size_t)(a.tiles_n + cur.tm) * op_half, op_half,
                       &bars->prep_full[buf]);
      }
    }
    __syncwarp();
  } else if (warp >= WT2_FIRST_EPI_WARP) {
    // ------------------------------ epilogue ----------------------------------
    // Two groups of eight warps; group grp owns the CTA's tiles i = grp, grp + 2, ... (accumulator stage i % 4,
    // operand buffer i % 2).  A thread is one weight row (TMEM lane) and one 64-column half of its group's
    // tile.  The groups meet only through the mbarriers.  While a group works on tile i the merge of its tile
    // i + 2 runs into the group's other accumulator stage, and with four W0 stages two loads are in flight.
    const int quarter = warp & 3;
    const int grp = (warp - WT2_FIRST_EPI_WARP) >> 3;
    const int chalf = ((warp - WT2_FIRST_EPI_WARP) >> 2) & 1;   // column half of the tile
    const int row = quarter * 32 + lane;
    const int tg = chalf * WT2_ROWS + row;                       // thread index within the group
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const int r = p.rank;
    const int L = a.n_opbuf;                                    // 1 or 2
    const int n_items = 32 * r;                                 // (row, 4 ranks) operand items per tile
    const int sbw = 2 * a.ngt;                                  // floats per thread: s x ngt | b x ngt
    float* grp_sb = sb_base + (size_t)grp * 2 * WT2_ROWS * sbw;   // two buffers of [128 rows][s x ngt | b x ngt]

    // ---- MMA operands of tile j (CTA sequence number), built by the group that owns the tile.  With two
    //      operand buffers the buffer of tile j was last read by the MMAs of tile j - 2, the group's own
    //      previous tile, which the caller has already seen complete; with one buffer by those of tile j - 1. ----
    auto prep_buffer_wait = [&](int j) {
      if (L == 1 && j >= 1) {
        bounded_wait(&bars->tmem_full[(j - 1) & 3], (uint32_t)(((j - 1) >> 2) & 1), bars);
        ptx::tc_fence_after_sync();
      }
    };
    auto prep = [&](int j, int m0_, int n0_) {
      if (a.op_img) return;                                     // warp 3 brings the operands in
      prep_buffer_wait(j);
      uint8_t* acat = op_base + (size_t)(j & (L - 1)) * 2 * op_half;
      for (int idx = tg; idx < n_items; idx += WT2_GROUP_THREADS) {
        OperandItem it_;
        operand_item_load(a, m0_, n0_, idx, it_);
        operand_item_store(a, idx, it_, acat, acat + op_half);
      }
      ptx::fence_proxy_async_smem();
      ptx::mbar_arrive(&bars->prep_full[j & (L - 1)]);
    };

    // ---- s and b of the tile's rows for the quantization groups it intersects: the threads of column half 0
    //      (one per weight row) copy them with asynchronous 4-byte copies into the group's buffer for its next
    //      tile; the group meets at a named barrier when it starts that tile.  (Each row's values sit in a line
    //      of their own, so every copy instruction touches 32 lines: the fewer of them the better.) ----
    auto stage_sb = [&](int m0_, int n0_, int buf) {
      if (chalf != 0 || a.sb_box) return;
      float* dst = grp_sb + ((size_t)buf * WT2_ROWS + row) * sbw;
      const int o_ = m0_ + row;
      const int gf = group_of(a, n0_);
      for (int k = 0; k < a.ngt; ++k) {
        const int g = gf + k;
        if (o_ < p.d_out && g < p.ngroups) {
          ptx::cp_async_4(dst + k, a.s + (size_t)o_ * p.ngroups + g);
          ptx::cp_async_4(dst + a.ngt + k, a.b + (size_t)o_ * p.ngroups + g);
        } else {
          dst[k] = 1.f; dst[a.ngt + k] = 0.f;
        }
      }
      ptx::cp_async_commit();
    };

    TileCursor cur(a, grp, WT2_GROUPS);
    if (cur.valid()) {
      stage_sb(cur.m0(), cur.n0(), 0);
      prep(grp, cur.m0(), cur.n0());
    }
    int sb_buf = 0;
    const int qn_bits = kRoundMagicBits + (int)p.qn;

    int stage = grp;                                            // W0 stage of tile i and its phase, kept without divisions
    uint32_t phase = 0;                                         // (n_stages >= 2 = WT2_GROUPS)
    for (int i = grp; cur.valid(); cur.next(), i += WT2_GROUPS) {
      const int m0 = cur.m0(), n0 = cur.n0();
      const int o = m0 + row;
      const bool row_ok = o < p.d_out;
      const int acc = i & 3;
      const int g_first = group_of(a, n0);
      int m1 = 0, n1 = 0;
      const bool has_next = cur.peek(1, m1, n1);
      const float *my_s, *my_b;                                 // s and b of this row, from group sb_first on
      int sb_first;
      if (a.sb_box) {                                           // they arrive with the W0 tile (full[stage] below)
        my_s = sb_base + ((size_t)stage * 2 * WT2_ROWS + row) * a.sb_box;
        my_b = my_s + WT2_ROWS * a.sb_box;
        sb_first = g_first & ~3;
      } else {
        ptx::cp_async_wait_all();                               // this thread's copies of the tile's s, b have landed
        ptx::named_bar_sync(1 + grp, WT2_GROUP_THREADS);        // ... and so have the group's
        my_s = grp_sb + ((size_t)sb_buf * WT2_ROWS + row) * sbw;
        my_b = my_s + a.ngt;
        sb_first = g_first;
      }
      bounded_wait(&bars->tmem_full[acc], (uint32_t)((i >> 2) & 1), bars);
      ptx::tc_fence_after_sync();
      // the merge of this tile is complete: the operands of the group's next tile can take its buffer
      if (has_next) prep(i + WT2_GROUPS, m1, n1);
      bounded_wait(&bars->full[stage], phase, bars);
      int ob = 0;
      if constexpr (HAS_OUT1) {
        const int uses = a.n_out == 2 ? (i >> 1) : i;           // earlier tiles that went through this buffer
        ob = a.n_out == 2 ? (i & 1) : 0;
        if (uses >= 1) bounded_wait(&bars->out_empty[ob], (uint32_t)((uses - 1) & 1), bars);
      }
      uint8_t* tile_rows = stage_base + (size_t)stage * WT2_STAGE_BYTES + row * 128;
      [[maybe_unused]] uint8_t* out1 = out_base + (size_t)ob * a.out_bytes;
      float rs = 1.f, s_ = 1.f, b_ = 0.f;
      int cur_g = -1;
#pragma unroll 1
      for (int bb = 0; bb < 2; ++bb) {                          // 32 columns
        const int blk = chalf * 2 + bb;
        [[maybe_unused]] uint32_t words[4] = {0u, 0u, 0u, 0u};  // WT2_PACK: the 32 codes of this block
#pragma unroll
        for (int half = 0; half < 2; ++half) {                  // 16 columns at a time
          uint32_t raw[16];
          ptx::tmem_ld_32x16(tmem_base + lane_base + (uint32_t)(acc * WT2_COLS + blk * 32 + half * 16), raw);
          ptx::tmem_ld_wait();
          if (bb == 1 && half == 1) {
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&bars->tmem_empty[acc]);
          }
#pragma unroll
          for (int s2 = 0; s2 < 2; ++s2) {
            const int sub = half * 2 + s2;
            const int piece = blk * 4 + sub;                    // 8-column piece of the tile (g % 8 == 0: one group)
            const int col = n0 + piece * 8;
            const bool ok = row_ok && col < p.d_in;
            const int g = group_of(a, col);
            const bool group_start = (col - g * p.group) == 0;
            if (g != cur_g) {                                   // one reciprocal per group
              cur_g = g;
              s_ = ok ? my_s[g - sb_first] : 1.f;
              b_ = ok ? my_b[g - sb_first] : 0.f;
              rs = 1.0f / s_;
            }
            const uint32_t chunk = (uint32_t)((piece >> 3) * (WT2_STAGE_BYTES / 2) + (((piece & 7) ^ (row & 7)) << 4));
            const uint4 wr = *reinterpret_cast<const uint4*>(tile_rows + chunk);
            const float w0[8] = {bf16_lo(wr.x), bf16_hi(wr.x), bf16_lo(wr.y), bf16_hi(wr.y),
                                 bf16_lo(wr.z), bf16_hi(wr.z), bf16_lo(wr.w), bf16_hi(wr.w)};
            float wq[8], fac[8];
            // Eq. 7-9 and the STE factor: the arithmetic of quantize_elem / ste_factor, with the rounding done
            // by the magic-number add (exact for the clamped range).  Two columns at a time on the packed fp32
            // pipe: every packed operation is the same IEEE operation per lane as its scalar form.
            const float2 gamma2 = make_float2(p.gamma, p.gamma), nb2 = make_float2(-b_, -b_), rs2 = make_float2(rs, rs);
            const float2 s2v = make_float2(s_, s_), b2v = make_float2(b_, b_);
            const float2 magic2 = make_float2(kRoundMagic, kRoundMagic), nmagic2 = make_float2(-kRoundMagic, -kRoundMagic);
#pragma unroll
            for (int e = 0; e < 8; e += 2) {
              const float2 acc2 = make_float2(__uint_as_float(raw[s2 * 8 + e]), __uint_as_float(raw[s2 * 8 + e + 1]));
              const float2 wc = __ffma2_rn(gamma2, acc2, make_float2(w0[e], w0[e + 1]));      // merge_elem
              const float2 w = __fmul2_rn(__fadd2_rn(wc, nb2), rs2);                         // (wc - b) * rs
              const float2 wcl = make_float2(fminf(fmaxf(w.x, p.qn), p.qp), fminf(fmaxf(w.y, p.qn), p.qp));
              const float2 y = __fadd2_rn(wcl, magic2);
              const float2 code = __fadd2_rn(y, nmagic2);
              const float2 q = __ffma2_rn(code, s2v, b2v);
              wq[e] = q.x; wq[e + 1] = q.y;
              if constexpr (MODE == WT2_DEQUANT_F) {
                const float2 t2 = __fadd2_rn(w, make_float2(-wcl.x, -wcl.y));                 // 0 inside [Q_N, Q_P]
                const float2 inr = __fadd2_rn(code, make_float2(-w.x, -w.y));                 // code - w
                const float tt[2] = {t2.x, t2.y}, ii[2] = {inr.x, inr.y};
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                  const float sentinel = __uint_as_float((__float_as_uint(tt[h]) & 0x80000000u) | 0x40000000u);   // +-2
                  fac[e + h] = (fabsf(tt[h]) > kMaskGuard) ? sentinel : ii[h];
                }
              }
              if constexpr (MODE == WT2_PACK) {                                     // code j of 32 at bit j * bits
                const float yy[2] = {y.x, y.y};
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                  const uint32_t u = (uint32_t)(__float_as_int(yy[h]) - qn_bits);
                  const int j = sub * 8 + e + h;
                  if (p.bits == 4) {
                    words[j >> 3] |= u << ((j & 7) * 4);
                  } else {
                    const int bit = j * 3, wd = bit >> 5, off = bit & 31;
                    words[wd] |= u << off;
                    if (off > 29) words[wd + 1] |= u >> (32 - off);
                  }
                }
              }
            }
            if constexpr (MODE != WT2_PACK) {
              uint4 o4;
              o4.x = pack_bf16x2(wq[0], wq[1]); o4.y = pack_bf16x2(wq[2], wq[3]);
              o4.z = pack_bf16x2(wq[4], wq[5]); o4.w = pack_bf16x2(wq[6], wq[7]);
              *reinterpret_cast<uint4*>(tile_rows + chunk) = o4;                    // in place, same swizzled position
            }
            if constexpr (MODE == WT2_DEQUANT_F) {
              __half2 h[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) h[e] = __floats2half2_rn(fac[2 * e], fac[2 * e + 1]);
              *reinterpret_cast<uint4*>(out1 + (piece * WT2_ROWS + row) * 16) = *reinterpret_cast<const uint4*>(h);
            }
            if constexpr (MODE == WT2_PACK) {
              if (ok && group_start) {                                              // first piece of its group
                a.s16[(size_t)o * p.ngroups + g] = __float2half_rn(s_);
                a.b16[(size_t)o * p.ngroups + g] = __float2half_rn(fmaf(s_, p.qn, b_));
              }
            }
          }
        }
        if constexpr (MODE == WT2_PACK) {
          // staging row = the tile's 128 codes of this weight row; this block is 32 of them
          if (p.bits == 4) {
            *reinterpret_cast<uint4*>(out1 + row * 64 + blk * 16) = make_uint4(words[0], words[1], words[2], words[3]);
          } else {
            uint32_t* dst = reinterpret_cast<uint32_t*>(out1 + row * 48 + blk * 12);
            dst[0] = words[0]; dst[1] = words[1]; dst[2] = words[2];
          }
        }
      }
      ptx::fence_proxy_async_smem();                   // the stores above are read by TMA
      ptx::mbar_arrive(&bars->written[stage]);
      sb_buf ^= 1;
      if (has_next) stage_sb(m1, n1, sb_buf);          // the other buffer: its readers passed this tile's barrier
      stage += WT2_GROUPS;
      if (stage >= a.n_stages) { stage -= a.n_stages; phase ^= 1; }
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

// uint32 row-major matrix [rows, words]; box = [box_words, box_rows], no swizzle (code words of the export).
inline bool make_tmap_words(CUtensorMap* m, const void* base, uint64_t rows, uint64_t words, uint32_t box_words,
                            uint32_t box_rows = 128) {
  PFN_encodeTiled enc = get_encode_fn();
  if (!enc) return false;
  const cuuint64_t gdim[2] = {words, rows};
  const cuuint64_t gstride[1] = {words * 4};
  const cuuint32_t box[2] = {box_words, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(base), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Shared-memory plan.  A tile being worked on holds one W0 stage and, when there is a second output, one
// staging buffer for it: two of each keep both epilogue groups busy, further stages let the loads run ahead.
// Candidates in order of preference (a single operand buffer makes every merge wait for the previous one).
// `sb_by_tma`: s and b may come in by TMA (the caller has checked their alignment); the shape must allow it too.
inline bool wtile_plan(WtileArgs& a, int mode, bool sb_by_tma = true) {
  const Params& p = a.p;
  a.atoms = (2 * p.rank + 31) / 32;
  a.ngt = std::min(p.ngroups, (WT2_COLS - 1) / p.group + 2);
  // a box starts at a group column that is a multiple of 4 (16 bytes) at or below the tile's first group, so it
  // is up to 3 groups wider than the tile; the row pitch of s and b must be a multiple of 16 bytes
  const int box = (a.ngt + 3 + 3) / 4 * 4;
  a.sb_box = (sb_by_tma && p.ngroups % 4 == 0 && p.ngroups >= box && box <= 256) ? box : 0;
  a.group_shift = -1;
  for (int sh = 3; sh < 31; ++sh)
    if ((1 << sh) == p.group) a.group_shift = sh;
  a.out_bytes = mode == WT2_DEQUANT_F ? WT2_STAGE_BYTES : mode == WT2_PACK ? WT2_ROWS * (WT2_COLS * p.bits / 8) : 0;
  struct Cand { int opbuf, n_out, stages; };
  static const Cand plain[] = {{2, 0, 4}, {1, 0, 4}, {2, 0, 3}, {1, 0, 3}, {2, 0, 2}, {1, 0, 2}};
  static const Cand small_out[] = {{2, 2, 4}, {1, 2, 4}, {2, 2, 3},
                                   {1, 2, 3}, {2, 2, 2}, {1, 2, 2}, {1, 1, 2}};
  static const Cand big_out[] = {{2, 2, 3}, {1, 2, 3}, {2, 2, 2}, {1, 2, 2}, {2, 1, 3}, {1, 1, 3},
                                 {2, 1, 2}, {1, 1, 2}};
  const Cand* cands = mode == WT2_DEQUANT ? plain : mode == WT2_PACK ? small_out : big_out;
  const int n_cands = mode == WT2_DEQUANT ? 6 : mode == WT2_PACK ? 7 : 8;
  const int max_opbuf = p.rank <= 32 ? 2 : 1;       // rank 64: the split operands of one tile are already 128 KB
  for (int c = 0; c < n_cands; ++c) {
    if (cands[c].opbuf > max_opbuf) continue;
    a.n_opbuf = cands[c].opbuf; a.n_out = cands[c].n_out; a.n_stages = cands[c].stages;
    if (wtile_smem_bytes(a) <= 227 * 1024) return true;
  }
  return false;
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
// Bytes of the operand images of a problem (see k_split_operands).
inline size_t wtile_image_bytes(const Params& p) {
  const size_t atoms = (2 * (size_t)p.rank + 31) / 32;
  return ((size_t)ceil_div(p.d_out, WT2_ROWS) + (size_t)ceil_div(p.d_in, WT2_COLS)) * atoms * WT2_ATOM_BYTES;
}

// `op_img` (optional, wtile_image_bytes(p) bytes of device scratch, 16-byte aligned): with it the MMA operands are
// split once by a launch of k_split_operands and reach the tiles by bulk copies; without it the epilogue warps
// build them tile by tile.  `zero` (optional): buffers that launch also clears; *zeroed is set when it did.
inline l4q_status launch_wtile_tc(int mode, const Params& p, const void* W0, const float* A, const float* B,
                                  const float* s, const float* b, void* out0, void* out1, __half* s16, __half* b16,
                                  cudaStream_t st, void* op_img = nullptr, const ZeroList* zero = nullptr,
                                  bool* zeroed = nullptr) {
  WtileArgs a{};
  a.p = p; a.A = A; a.B = B; a.s = s; a.b = b; a.s16 = s16; a.b16 = b16;
  a.tiles_m = ceil_div(p.d_out, WT2_ROWS);
  a.tiles_n = ceil_div(p.d_in, WT2_COLS);
  const bool sb_aligned = ((reinterpret_cast<uintptr_t>(s) | reinterpret_cast<uintptr_t>(b)) & 15u) == 0;
  if (!wtile_plan(a, mode, sb_aligned)) return L4Q_ERR_UNSUPPORTED;
  CUtensorMap t_w0, t_o0, t_o1, t_s, t_b;
  if (!make_tmap_bf16(&t_w0, W0, p.d_out, p.d_in, WT2_ROWS)) return L4Q_ERR_CUDA;
  t_o1 = t_w0;
  if (mode == WT2_PACK) {
    if (!make_tmap_words(&t_o0, out0, p.d_out, ((uint64_t)p.d_in * p.bits) >> 5, WT2_COLS * p.bits / 32))
      return L4Q_ERR_CUDA;
  } else {
    if (!make_tmap_bf16(&t_o0, out0, p.d_out, p.d_in, WT2_ROWS)) return L4Q_ERR_CUDA;
    a.F = reinterpret_cast<__half*>(out1);
  }
  t_s = t_w0; t_b = t_w0;                          // placeholders when unused
  if (a.sb_box) {                                   // fp32 moved as 32-bit words
    if (!make_tmap_words(&t_s, s, p.d_out, p.ngroups, a.sb_box) || !make_tmap_words(&t_b, b, p.d_out, p.ngroups, a.sb_box))
      return L4Q_ERR_CUDA;
  }
  const size_t smem = wtile_smem_bytes(a);
  const int grid = std::min(a.tiles_m * a.tiles_n, sm_count());
  if (op_img) {
    ZeroList zl{};
    if (zero) zl = *zero;
    k_split_operands<<<a.tiles_n + a.tiles_m, 256, 0, st>>>(a, static_cast<uint8_t*>(op_img), zl);
    if (cudaGetLastError() != cudaSuccess) return L4Q_ERR_CUDA;
    if (zero && zeroed) *zeroed = true;
    a.op_img = static_cast<const uint8_t*>(op_img);
  }
  auto launch = [&](auto kern) -> l4q_status {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return L4Q_ERR_CUDA;
    kern<<<grid, WT2_THREADS, smem, st>>>(t_w0, t_o0, t_o1, t_s, t_b, a);
    return cudaGetLastError() == cudaSuccess ? L4Q_OK : L4Q_ERR_CUDA;
  };
  switch (mode) {
    case WT2_DEQUANT: return launch(k_wtile_tc<WT2_DEQUANT>);
    case WT2_DEQUANT_F: return launch(k_wtile_tc<WT2_DEQUANT_F>);
    default: return launch(k_wtile_tc<WT2_PACK>);
  }
}

}  // namespace l4q
