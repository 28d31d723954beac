// Weight-tile kernel of the bf16 path: merge (Eq. 7) + fake-quantize (Eq. 8-9) the weight in
// 128 x 128 tiles, streaming W0 once from HBM, and write one of
//   WT2_DEQUANT    W_q (bf16)                      -- the recompute step of forward and backward (App. E.2)
//   WT2_DEQUANT_F  W_q (bf16) + STE factors (fp16) -- backward: input gradient + weight-gradient reduction
//                  (the factors leave from registers, 16 bytes per thread and 8-column piece, coalesced)
//   WT2_PACK       bit-packed codes + fp16 s, b    -- export (Sec. 3.2)
//   WT2_FACTORS    STE factors alone               -- backward without the input gradient: W_q is not needed
//   WT2_ERROR      E_quant, E_clip (two sums)      -- the quantization-error metric of Table 4; nothing else is written
//
// HBM-bound by design (2 bytes in, 0.4-4 bytes out per weight), so everything else is arranged to stay out
// of the way of the copies:
//   * W0 tiles arrive by TMA into 128-byte-swizzled shared memory (up to 5 stages in flight); W_q is written
//     back IN PLACE into the same stage and leaves by a TMA store, so every global access is a full line;
//   * the rank-r merge B A is a tensor-core contraction: tcgen05.mma kind::tf32 into tensor memory, with
//     each fp32 factor split into a tf32 head and a tf32 tail (x = hi + lo, three products hi*hi + hi*lo +
//     lo*hi), which keeps ~21 mantissa bits -- the codes must agree with fp64 arithmetic except within
//     1e-6 of a rounding boundary, which a single tf32 or bf16 product does not give;
//   * the MMA operands of the merge (the tile's slices of A and B, each value split into head / tail, K-major
//     with the 128-byte swizzle) are written once per launch for every column and row panel by
//     k_split_operands, laid out as they stand in shared memory.  A CTA works on a contiguous run of the
//     column-panel-major tile sequence, so the A image of its column panel stays resident (reloaded at a panel
//     change) and only the B image of the tile's row panel streams in, 16 KB (one swizzle atom of K) at a
//     time through a ring of chunks, each released by the MMAs that read it;
//   * 16 epilogue warps in two groups of eight; a group owns every second tile of the CTA (accumulator stage
//     tile % 4), a thread one weight row and one 64-column half of the group's tile.  It reads the
//     merge from tensor memory with tcgen05.ld, the W0 tile from shared memory in 16-byte pieces, and does
//     the quantizer arithmetic.  Interior tiles whose half rows lie in one quantization
//     group take wtile_half_row_fast (no per-element bounds or group logic; s and b come straight from
//     global memory, one pair per thread and tile, fetched a tile ahead); every other tile takes the
//     general loop.
//
// Roles (672 threads): warp 0 = TMA loads (W0; s, b boxes where used), warp 1 = MMA issuer + TMEM owner,
// warps 2 and 20 = TMA stores (one thread each, alternate tiles), warp 3 = operand loader (one thread issuing bulk copies of the ready-made images, or,
// without images, the whole warp building the operands from A and B), warps 4..19 = epilogue (warp w: TMEM
// lane quarter w % 4, group (w - 4) / 8, column half ((w - 4) / 4) % 2).
// Every mbarrier wait is bounded (see bounded_wait); there is no block-level barrier after set-up.
#pragma once

#include "l4q_common.cuh"
#include "l4q_gemm.cuh"
#include "l4q_ptx.cuh"

namespace l4q {

constexpr int WT2_ROWS = 128, WT2_COLS = 128;
#ifndef WT2_NGROUPS
#define WT2_NGROUPS 2
#endif
constexpr int WT2_THREADS = 128 + 256 * WT2_NGROUPS + 32;   // four role warps, the epilogue groups, the second store warp
constexpr int WT2_FIRST_EPI_WARP = 4;
constexpr int WT2_SECOND_STORE_WARP = WT2_FIRST_EPI_WARP + 8 * WT2_NGROUPS;
constexpr int WT2_BUILDERS = 32;                    // threads that build the merge operands where no images are given: warp 3
                                                    // (four warps were measured too: still far slower than ready-made images)
constexpr int WT2_EPI_THREADS = 256 * WT2_NGROUPS;
constexpr int WT2_GROUPS = WT2_NGROUPS;                       // epilogue warp groups; group g owns tiles g, g + WT2_GROUPS, ... of the CTA
constexpr int WT2_GROUP_THREADS = WT2_EPI_THREADS / WT2_GROUPS;
constexpr int WT2_ACC = 4;                          // accumulator stages of 128 TMEM columns
constexpr int WT2_STAGE_BYTES = WT2_ROWS * WT2_COLS * 2;   // one bf16 tile: two 128 x 64 swizzled boxes
constexpr int WT2_ATOM_BYTES = 128 * 128;           // 128 rows x 32 tf32 (one 128-byte swizzle atom along K)
constexpr int WT2_MAX_STAGES = 6;
constexpr int WT2_MAX_BSLOTS = 8;
constexpr int WT2_MAX_ATOMS = 4;                    // rank <= 64

enum { WT2_DEQUANT = 0, WT2_DEQUANT_F = 1, WT2_PACK = 2, WT2_ERROR = 3, WT2_FACTORS = 4 };
__host__ __device__ constexpr bool wt2_has_factors(int mode) { return mode == WT2_DEQUANT_F || mode == WT2_FACTORS; }
__host__ __device__ constexpr bool wt2_has_wq(int mode) { return mode == WT2_DEQUANT || mode == WT2_DEQUANT_F; }

// Output buffers of the caller that must start from zero (they are accumulated into with atomics later on the
// stream): cleared by a launch that runs anyway, which saves one memset launch per buffer.
struct ZeroList { float* ptr[4]; size_t n[4]; };

// bf16 copies of the LoRA factors for the weight-gradient kernel of the same backward call, which contracts its
// G * m tiles with them on the tensor cores (Eq. 13-14): A16 [rn, d_in] and Bt16 = B^T [rn, d_out], row-major,
// rows beyond the rank zero (rn = the MMA's N, a multiple of 16).  Written by the operand-split launch.
struct Bf16Copies {
  __nv_bfloat16 *A16, *Bt16;
  int rn;
};

struct WtileArgs {
  Params p;
  const float *A, *B, *s, *b;
  __half *s16, *b16;       // WT2_PACK
  __half* F;               // WT2_DEQUANT_F: the factor array (factor_index layout)
  double* errors;          // WT2_ERROR: E_quant, E_clip (accumulated with fp64 atomics; zero on entry)
  ZeroList zero;           // buffers this launch clears before anything else (all sizes 0: none)
  const uint8_t* op_img;   // optional: the split MMA operands of every panel, ready made (see k_split_operands)
  int tiles_m, tiles_n;
  int n_stages;            // W0 stages in shared memory (2..5)
  int n_out;               // staging buffers for the code words of the export: one per epilogue group (0 in other modes)
  int out_bytes;           // bytes of one such buffer
  int atoms;               // swizzle atoms per operand row: ceil(2 rank / 32)
  int ngt;                 // upper bound of the quantization groups a 128-column tile intersects
  int n_abuf;              // buffers for the A image of a column panel (atoms x 16 KB each): 1 or 2
  int n_bslot;             // ring of 16 KB chunks of the B images
  int group_shift;         // log2(group size) if it is a power of two, else -1
  int fast;                // interior tiles take wtile_half_row_fast (group a multiple of 64); s and b are then read
                           // from global memory and no copy of them is staged in shared memory
  int sb_box;              // groups per row of the s / b boxes that TMA brings in with the W0 tile; 0: none
};

// column / group size without a division in the common power-of-two case
__device__ __forceinline__ int group_of(const WtileArgs& a, int col) {
  return a.group_shift >= 0 ? (col >> a.group_shift) : (col / a.p.group);
}

struct __align__(8) WtileBarriers {
  uint64_t full[WT2_MAX_STAGES];      // W0 tile has landed in the stage
  uint64_t empty[WT2_MAX_STAGES];     // the stage may be overwritten (its store has read it)
  uint64_t written[WT2_MAX_STAGES];   // the epilogue has written the stage's outputs
  uint64_t out_empty[WT2_GROUPS];     // staging buffer of the code words may be overwritten
  uint64_t afull[2], aempty[2];       // A image of a column panel: complete in buffer b / no longer read by any MMA
  uint64_t bfull[WT2_MAX_BSLOTS], bempty[WT2_MAX_BSLOTS];   // one chunk of a B image, likewise
  uint64_t tmem_full[WT2_ACC], tmem_empty[WT2_ACC];
  uint32_t tmem_base;
  volatile uint32_t abort;
};

// s and b staged in shared memory by the epilogue warps (general path without TMA boxes): per epilogue thread
// [s x ngt | b x ngt] floats of its weight row; a thread reads and writes its own entry only.
__host__ __device__ inline size_t wtile_sb_bytes(int ngt) { return (size_t)WT2_EPI_THREADS * 2 * ngt * sizeof(float); }

// With sb_box: per W0 stage one box [128 rows][sb_box] of s and one of b.  On the fast path: nothing.
__host__ __device__ inline size_t wtile_sb_region_bytes(const WtileArgs& a) {
  if (a.fast) return 0;
  return a.sb_box ? (size_t)a.n_stages * 2 * WT2_ROWS * a.sb_box * sizeof(float) : wtile_sb_bytes(a.ngt);
}
inline size_t wtile_smem_bytes(const WtileArgs& a) {
  return 1024 + (size_t)a.n_stages * WT2_STAGE_BYTES + (size_t)a.n_out * a.out_bytes +
         ((size_t)a.n_abuf * a.atoms + a.n_bslot) * WT2_ATOM_BYTES + wtile_sb_region_bytes(a) + sizeof(WtileBarriers);
}

// The tiles of one CTA: a contiguous run [t0, t1) of the column-panel-major sequence (row tiles of one column
// panel are consecutive), runs of equal length up to one tile, so that the A image of a column panel is loaded
// once or twice per CTA.  (Handing tiles out strided by the grid size, neighbouring CTAs on neighbouring row
// tiles, was measured and made no difference to the memory system.)  Coordinates advance without divisions.
struct TileCursor {
  int t, t1, tm, tn, tiles_m, step;
  // the run's tiles number first, first + stride, ...
  __device__ explicit TileCursor(const WtileArgs& a, int first = 0, int stride = 1) {
    const long long total = (long long)a.tiles_m * a.tiles_n;
    tiles_m = a.tiles_m;
    t = (int)(total * blockIdx.x / gridDim.x) + first;
    t1 = (int)(total * (blockIdx.x + 1) / gridDim.x);
    tn = t / tiles_m; tm = t - tn * tiles_m;
    step = stride;
  }
  __device__ bool valid() const { return t < t1; }
  __device__ void next() {
    t += step; tm += step;
    while (tm >= tiles_m) { tm -= tiles_m; ++tn; }
  }
  __device__ int m0() const { return tm * WT2_ROWS; }
  __device__ int n0() const { return tn * WT2_COLS; }
  // coordinates of the run's tile k (small) steps ahead; false beyond the end
  __device__ bool peek(int k, int& m0_, int& n0_) const {
    if (t + k * step >= t1) return false;
    int m = tm + k * step, n = tn;
    while (m >= tiles_m) { m -= tiles_m; ++n; }
    m0_ = m * WT2_ROWS; n0_ = n * WT2_COLS;
    return true;
  }
};

// The W0 stages (and, in the export, the staging buffers of the code words) are owned by the epilogue groups:
// group g works through stages g, g + G, g + 2 G, ... of the n_stages, round after round.  Every barrier of a
// stage then has one waiting thread per side, which sees its phases strictly in order -- a barrier that two
// threads waited on in turn, a whole round of stages apart, could be taken for complete one phase early by the
// parity test whenever the groups had drifted three tiles apart.
struct StageSeq {
  int g, n_own, slot, round;
  __device__ StageSeq(int group, int n_stages) : g(group), slot(0), round(0) {
    n_own = (n_stages - group + WT2_GROUPS - 1) / WT2_GROUPS;          // stages g, g + G, ... below n_stages
  }
  __device__ int stage() const { return g + WT2_GROUPS * slot; }
  __device__ uint32_t parity() const { return (uint32_t)(round & 1); }
  __device__ void advance() { if (++slot == n_own) { slot = 0; ++round; } }
};

// x = hi + lo with hi, lo representable in tf32 (low 13 mantissa bits clear): hi keeps the leading 10
// mantissa bits of x (truncation), lo the leading bits of the exact remainder.  Plain logic ops.
__device__ __forceinline__ void split_tf32(float x, float& hi, float& lo) {
  hi = __uint_as_float(__float_as_uint(x) & 0xFFFFE000u);
  lo = __uint_as_float(__float_as_uint(x - hi) & 0xFFFFE000u);
}

// MMA operands of one tile, K-major with the 128-byte swizzle, one atom (32 values of K, 16 KB) at a time:
//   A image, row n = column n0 + n of the weight:  [ hi(A[0..r, col]) | lo(A[0..r, col]) ]
//   B image, row m = row m0 + m of the weight:      [ hi(B[row, 0..r]) | lo(B[row, 0..r]) ]
// Atom c holds values 32 c .. 32 c + 31 of that concatenation (beyond 2 r: zero).  A work item is one 16-byte
// piece (4 values) of one row: item it -> row it % 128, piece it / 128, so that a warp reads 32 consecutive
// columns of A (coalesced) or 32 rows of B.  `dst`: the atom, in shared or global memory.
// NT threads take 1024 / NT items each, in batches of up to 8 whose loads are all issued before the first is used.
template <int NT>
__device__ __forceinline__ void build_atom_a(const WtileArgs& a, int n0, int c, uint8_t* dst, int tid) {
  const Params& p = a.p;
  constexpr int PER = 1024 / NT, BATCH = PER < 8 ? PER : 8;
#pragma unroll 1
  for (int u0 = 0; u0 < PER; u0 += BATCH) {
    float x[BATCH][4];
#pragma unroll
    for (int u = 0; u < BATCH; ++u) {
      const int it = tid + (u0 + u) * NT, row = it & 127, j = it >> 7, e0 = 32 * c + 4 * j, col = n0 + row;
      const int k = e0 >= p.rank ? e0 - p.rank : e0;
      const bool ok = e0 < 2 * p.rank && col < p.d_in;
#pragma unroll
      for (int e = 0; e < 4; ++e) x[u][e] = ok ? __ldg(a.A + (size_t)(k + e) * p.d_in + col) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < BATCH; ++u) {
      const int it = tid + (u0 + u) * NT, row = it & 127, j = it >> 7, e0 = 32 * c + 4 * j;
      const bool tail = e0 >= p.rank;
      float h[4], l[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) split_tf32(x[u][e], h[e], l[e]);
      *reinterpret_cast<float4*>(dst + row * 128 + ((j ^ (row & 7)) << 4)) =
          tail ? make_float4(l[0], l[1], l[2], l[3]) : make_float4(h[0], h[1], h[2], h[3]);
    }
  }
}

template <int NT>
__device__ __forceinline__ void build_atom_b(const WtileArgs& a, int m0, int c, uint8_t* dst, int tid) {
  const Params& p = a.p;
  constexpr int PER = 1024 / NT, BATCH = PER < 8 ? PER : 8;
#pragma unroll 1
  for (int u0 = 0; u0 < PER; u0 += BATCH) {
    float4 x[BATCH];
#pragma unroll
    for (int u = 0; u < BATCH; ++u) {
      const int it = tid + (u0 + u) * NT, row = it & 127, j = it >> 7, e0 = 32 * c + 4 * j, o = m0 + row;
      const int k = e0 >= p.rank ? e0 - p.rank : e0;
      x[u] = (e0 < 2 * p.rank && o < p.d_out) ? __ldg(reinterpret_cast<const float4*>(a.B + (size_t)o * p.rank + k))
                                              : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < BATCH; ++u) {
      const int it = tid + (u0 + u) * NT, row = it & 127, j = it >> 7, e0 = 32 * c + 4 * j;
      const bool tail = e0 >= p.rank;
      const float v[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
      float h[4], l[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) split_tf32(v[e], h[e], l[e]);
      *reinterpret_cast<float4*>(dst + row * 128 + ((j ^ (row & 7)) << 4)) =
          tail ? make_float4(l[0], l[1], l[2], l[3]) : make_float4(h[0], h[1], h[2], h[3]);
    }
  }
}

// The operand images of all panels, written once per launch of the weight-tile kernel: image tn (tn < tiles_n)
// is the A image of column panel tn, image tiles_n + tm the B image of row panel tm, each `atoms` atoms exactly
// as they stand in shared memory, so that bulk copies bring them in.  One block per quarter of an atom, one
// 16-byte piece per thread: the launch is short, and the kernel that follows waits for it.
__global__ void __launch_bounds__(256) k_split_operands(const WtileArgs a, uint8_t* __restrict__ img, int image_blocks,
                                                        const Bf16Copies cp) {
  // the weight-tile kernel that follows may start now: it loads W0 tiles while the images are being written and
  // waits for this grid (griddep_wait) only before it copies the first image
  ptx::griddep_launch_dependents();
  const Params& p = a.p;
  if ((int)blockIdx.x >= image_blocks) {
    // the blocks after the images: bf16 copies of A and of B^T, 8 values per thread
    const long long e = ((long long)(blockIdx.x - image_blocks) * 256 + threadIdx.x) * 8;
    const long long na = (long long)cp.rn * p.d_in, nb = (long long)cp.rn * p.d_out;
    float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    __nv_bfloat16* dst = nullptr;
    if (e < na) {                                    // A16[k, col .. col + 7]   (d_in is a multiple of 8)
      const int k = (int)(e / p.d_in), col = (int)(e - (long long)k * p.d_in);
      if (k < p.rank) {
        const float4 x0 = __ldg(reinterpret_cast<const float4*>(a.A + (size_t)k * p.d_in + col));
        const float4 x1 = __ldg(reinterpret_cast<const float4*>(a.A + (size_t)k * p.d_in + col + 4));
        v[0] = x0.x; v[1] = x0.y; v[2] = x0.z; v[3] = x0.w; v[4] = x1.x; v[5] = x1.y; v[6] = x1.z; v[7] = x1.w;
      }
      dst = cp.A16 + e;
    } else if (e - na < nb) {                        // Bt16[k, o .. o + 7]      (d_out is a multiple of 8)
      const long long f = e - na;
      const int k = (int)(f / p.d_out), o = (int)(f - (long long)k * p.d_out);
      if (k < p.rank) {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = __ldg(a.B + (size_t)(o + j) * p.rank + k);
      }
      dst = cp.Bt16 + f;
    }
    if (dst) {
      uint4 o4;
      o4.x = pack_bf16x2(v[0], v[1]); o4.y = pack_bf16x2(v[2], v[3]);
      o4.z = pack_bf16x2(v[4], v[5]); o4.w = pack_bf16x2(v[6], v[7]);
      *reinterpret_cast<uint4*>(dst) = o4;
    }
    return;
  }
  const int quarter = blockIdx.x & 3, c = (blockIdx.x >> 2) % a.atoms, panel = (blockIdx.x >> 2) / a.atoms;
  uint8_t* dst = img + ((size_t)panel * a.atoms + c) * WT2_ATOM_BYTES;
  const int it = quarter * 256 + threadIdx.x, row = it & 127, j = it >> 7, e0 = 32 * c + 4 * j;
  const bool tail = e0 >= p.rank;
  const int k = tail ? e0 - p.rank : e0;
  float x[4] = {0.f, 0.f, 0.f, 0.f};
  if (e0 < 2 * p.rank) {
    if (panel < a.tiles_n) {
      const int col = panel * WT2_COLS + row;
      if (col < p.d_in) {
#pragma unroll
        for (int e = 0; e < 4; ++e) x[e] = __ldg(a.A + (size_t)(k + e) * p.d_in + col);
      }
    } else {
      const int o = (panel - a.tiles_n) * WT2_ROWS + row;
      if (o < p.d_out) {
        const float4 bv = __ldg(reinterpret_cast<const float4*>(a.B + (size_t)o * p.rank + k));
        x[0] = bv.x; x[1] = bv.y; x[2] = bv.z; x[3] = bv.w;
      }
    }
  }
  float h[4], l[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) split_tf32(x[e], h[e], l[e]);
  *reinterpret_cast<float4*>(dst + row * 128 + ((j ^ (row & 7)) << 4)) =
      tail ? make_float4(l[0], l[1], l[2], l[3]) : make_float4(h[0], h[1], h[2], h[3]);
}

// Adding and subtracting 1.5 * 2^23 rounds |x| < 2^22 to the nearest integer, ties to even, exactly like
// rintf, on the FP32 add pipe; the low mantissa bits of the intermediate sum hold that integer.
constexpr float kRoundMagic = 12582912.0f;
constexpr int kRoundMagicBits = 0x4B400000;

// The merge MMAs of one B chunk (atom c of the tile's B image, at shared address `bchunk`) against the resident
// A image at `acat`:  B A = Bhi Ahi + Bhi Alo + Blo Ahi  (the tail x tail product is below fp32 resolution of
// the sum).  A K step is 8 values (32 bytes); a head step of B meets the head and the tail of A, a tail step
// the head of A.  `first` : the tile's first MMA overwrites the accumulator.  With R known at compile time the
// whole sequence is straight-line code: the issuing thread shares its scheduler with four epilogue warps, and
// every instruction of a data-dependent address computation costs it several cycles.
__device__ __forceinline__ uint64_t wt_desc(uint32_t lo_base, uint32_t byte_off) {
  constexpr uint32_t HI = ((1024u >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);   // SBO 1024, version 1, 128-byte swizzle
  return ((uint64_t)HI << 32) | (lo_base + (byte_off >> 4));
}
__device__ __forceinline__ uint32_t wt_desc_lo(uint32_t smem_addr) {
  return ((smem_addr >> 4) & 0x3FFFu) | (1u << 16);                            // start address, LBO 16 bytes
}
// byte offset of value e of an image row inside the image (atom, then position in the 128-byte row)
__host__ __device__ constexpr uint32_t wt_elem_off(int e) { return (uint32_t)(e >> 5) * WT2_ATOM_BYTES + (uint32_t)(e & 31) * 4u; }

template <int R>
__device__ __forceinline__ void issue_chunk_mmas(int c, int rank, uint32_t bchunk, uint32_t acat, uint32_t d_tmem) {
  constexpr uint32_t idesc = ptx::make_idesc_tf32(WT2_ROWS, WT2_COLS);
  const uint32_t b_lo = wt_desc_lo(bchunk), a_lo = wt_desc_lo(acat);
  const int r = R > 0 ? R : rank;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int e = 32 * c + 8 * k;                    // value index in the B row
    if (e >= 2 * r) break;
    const uint64_t dm = wt_desc(b_lo, (uint32_t)k * 32u);
    if (e < r) {
      ptx::mma_tf32_ss(d_tmem, dm, wt_desc(a_lo, wt_elem_off(e)), idesc, e != 0 ? 1u : 0u);
      ptx::mma_tf32_ss(d_tmem, dm, wt_desc(a_lo, wt_elem_off(r + e)), idesc, 1u);
    } else {
      ptx::mma_tf32_ss(d_tmem, dm, wt_desc(a_lo, wt_elem_off(e - r)), idesc, 1u);
    }
  }
}

// ---------------------------------------------------------------------------
// Epilogue arithmetic of an interior tile whose half rows (64 columns of one weight row) lie inside one
// quantization group: the arithmetic of quantize_elem / ste_factor, element for element the same operations in
// the same order as everywhere else in the library (so that every kernel takes the same rounding and gating
// decisions, ties included), without bounds tests or group bookkeeping per element, two columns at a time on
// the packed fp32 pipe, with the rounding done by the magic-number add (exact for the clamped range).
// ---------------------------------------------------------------------------

// Sum over j < n of (1.5 * 2^23 as bits) << (j * bits), modulo 2^32: what the magic-number bit patterns add up to
// when n raw y words are accumulated at their bit offsets instead of the bare codes.
__host__ __device__ constexpr uint32_t magic_bias(int n, int bits) {
  uint32_t k = 0;
  for (int j = 0; j < n; ++j) k += (j * bits < 32) ? ((uint32_t)0x4B400000u << (j * bits)) : 0u;
  return k;
}

// Per-thread constants of a tile on the fast path.
struct FastConsts {
  float s, b, rs;        // rs = 1 / s
  float qn, qp, gamma;
};

// One half row (64 columns) of an interior tile.  `taddr`: TMEM address of the thread's first merge column;
// `tile_row`: the thread's row of the W0 stage (swizzled; pieces of 16 bytes).  MODE WT2_DEQUANT /
// WT2_DEQUANT_F: W_q overwrites W0 in place, the factors go to `out1` (the tile's block of the factor array);
// WT2_PACK (unsigned grid only): the code words go to `out1` (the tile's staging rows).
template <int MODE, int BITS>
__device__ __forceinline__ void wtile_half_row_fast(const FastConsts& c, uint32_t taddr, uint8_t* tile_row, int row,
                                                    int chalf, uint8_t* out1, uint64_t* tmem_empty_bar,
                                                    float& e_quant, float& e_clip) {
  const float2 gamma2 = make_float2(c.gamma, c.gamma), nb2 = make_float2(-c.b, -c.b), rs2 = make_float2(c.rs, c.rs);
  const float2 magic2 = make_float2(kRoundMagic, kRoundMagic);
  [[maybe_unused]] const float2 nmagic2 = make_float2(-kRoundMagic, -kRoundMagic);
  [[maybe_unused]] const float2 s2v = make_float2(c.s, c.s), b2v = make_float2(c.b, c.b);
  [[maybe_unused]] uint32_t words[4];                                           // BITS == 4: four words = 32 codes
  [[maybe_unused]] uint32_t h3[3] = {0u, 0u, 0u}, carry10 = 0u, carry21 = 0u;   // BITS == 3: 32 codes -> 3 words
  // The 64 columns in two rounds of 32 (a loop, not unrolled: the straight-line code of all 64 is several times
  // the instruction cache of a scheduler, and two groups run it at different places), each round two TMEM loads
  // of 16 columns, the second in flight while the first is worked on.
#pragma unroll 1
  for (int hq = 0; hq < 2; ++hq) {
  uint32_t raw[2][16];
  ptx::tmem_ld_32x16(taddr + (uint32_t)(hq * 32), raw[0]);
#pragma unroll
  for (int ql = 0; ql < 2; ++ql) {                    // 16 columns
    ptx::tmem_ld_wait();
    if (ql == 0) {
      ptx::tmem_ld_32x16(taddr + (uint32_t)(hq * 32 + 16), raw[1]);
    } else if (hq == 1) {                             // all of the thread's merge columns are in registers
      ptx::tc_fence_before_sync();
      ptx::mbar_arrive(tmem_empty_bar);
    }
    const uint32_t(&acc)[16] = raw[ql];
#pragma unroll
    for (int s2 = 0; s2 < 2; ++s2) {
      const int pl = ql * 2 + s2;                     // piece of the round (static), of the half row:
      const int pin = hq * 4 + pl;
      const int piece = chalf * 8 + pin;              // piece of the tile row (chalf selects the 64-column box)
      const uint32_t chunk = (uint32_t)((piece >> 3) * (WT2_STAGE_BYTES / 2) + (((piece & 7) ^ (row & 7)) << 4));
      const uint4 wr = *reinterpret_cast<const uint4*>(tile_row + chunk);
      const uint32_t wv[4] = {wr.x, wr.y, wr.z, wr.w};
      [[maybe_unused]] uint32_t qo[4];
      [[maybe_unused]] uint32_t fo[4];
      [[maybe_unused]] uint32_t word4 = 0u;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 acc2 = make_float2(__uint_as_float(acc[s2 * 8 + 2 * e]), __uint_as_float(acc[s2 * 8 + 2 * e + 1]));
        const float2 wc = __ffma2_rn(gamma2, acc2, make_float2(bf16_lo(wv[e]), bf16_hi(wv[e])));
        const float2 w = __fmul2_rn(__fadd2_rn(wc, nb2), rs2);                     // (wc - b) * rs
        const float2 wcl = make_float2(fminf(fmaxf(w.x, c.qn), c.qp), fminf(fmaxf(w.y, c.qn), c.qp));
        const float2 y = __fadd2_rn(wcl, magic2);
        if constexpr (MODE != WT2_PACK) {
          const float2 code = __fadd2_rn(y, nmagic2);
          const float2 wq = __ffma2_rn(code, s2v, b2v);
          qo[e] = pack_bf16x2(wq.x, wq.y);
          if constexpr (MODE == WT2_ERROR) {                                       // |W_comb - W_q|, and its part outside the range
            const float2 t2 = __fadd2_rn(w, make_float2(-wcl.x, -wcl.y));
            const float ex = fabsf(wc.x - wq.x), ey = fabsf(wc.y - wq.y);
            e_quant += ex + ey;
            e_clip += (fabsf(t2.x) > kMaskGuard ? ex : 0.f) + (fabsf(t2.y) > kMaskGuard ? ey : 0.f);
          }
          if constexpr (wt2_has_factors(MODE)) {
            const float2 t2 = __fadd2_rn(w, make_float2(-wcl.x, -wcl.y));          // 0 inside [Q_N, Q_P]
            const float2 inr = __fadd2_rn(code, make_float2(-w.x, -w.y));          // w~ - w
            const float tt[2] = {t2.x, t2.y}, ii[2] = {inr.x, inr.y};
            float f[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const float sentinel = __uint_as_float((__float_as_uint(tt[h]) & 0x80000000u) | 0x40000000u);   // +-2
              f[h] = (fabsf(tt[h]) > kMaskGuard) ? sentinel : ii[h];
            }
            const __half2 hh = __floats2half2_rn(f[0], f[1]);
            fo[e] = *reinterpret_cast<const uint32_t*>(&hh);
          }
        } else {
          const uint32_t yb[2] = {__float_as_uint(y.x), __float_as_uint(y.y)};
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            if constexpr (BITS == 4) {
              const int j = 2 * e + h;                                           // code j of the word at bit 4 j
              word4 = (j == 0) ? yb[h] : word4 + (yb[h] << (4 * j));
            } else {
              const int j = pl * 8 + 2 * e + h;                                  // code j of 32 at bit 3 j of 3 words
              if (j < 10) h3[0] += yb[h] << (3 * j);
              else if (j == 10) carry10 = yb[h] & 7u;
              else if (j < 21) h3[1] += yb[h] << (3 * (j - 11) + 1);
              else if (j == 21) carry21 = yb[h] & 7u;
              else h3[2] += yb[h] << (3 * (j - 22) + 2);
            }
          }
        }
      }
      if constexpr (wt2_has_wq(MODE))
        *reinterpret_cast<uint4*>(tile_row + chunk) = make_uint4(qo[0], qo[1], qo[2], qo[3]);   // in place
      if constexpr (wt2_has_factors(MODE))
        *reinterpret_cast<uint4*>(out1 + (piece * WT2_ROWS + row) * 16) = make_uint4(fo[0], fo[1], fo[2], fo[3]);
      // staging row = the tile's 128 codes of this weight row; this thread writes 64 of them, 32 at a time
      if constexpr (MODE == WT2_PACK && BITS == 4) {
        words[pl] = word4 - magic_bias(8, 4);
        if (pl == 3)
          *reinterpret_cast<uint4*>(out1 + row * 64 + chalf * 32 + hq * 16) =
              make_uint4(words[0], words[1], words[2], words[3]);
      }
      if constexpr (MODE == WT2_PACK && BITS == 3) {
        if (pl == 3) {
          uint32_t* dst = reinterpret_cast<uint32_t*>(out1 + row * 48 + chalf * 24 + hq * 12);
          dst[0] = (h3[0] - magic_bias(10, 3)) + (carry10 << 30);
          dst[1] = (h3[1] - (magic_bias(10, 3) << 1)) + (carry10 >> 2) + (carry21 << 31);
          dst[2] = (h3[2] - (magic_bias(10, 3) << 2)) + (carry21 >> 1);
          h3[0] = h3[1] = h3[2] = 0u;
        }
      }
    }
  }
  }
}

// The MMA issuer of the weight-tile kernel: one thread.  It shares its warp scheduler with four epilogue warps, so
// every instruction here waits its turn: the loop is kept to the barrier polls, the MMAs with descriptors that
// differ from precomputed ones by constants, and the tile cursor (no flag reads: a wait that gives up reports it).
template <int R>
__device__ __forceinline__ void wtile_mma_role(const WtileArgs& a, WtileBarriers* bars, uint32_t tmem_base,
                                               uint32_t acat_addr, uint32_t bslot_addr) {
  TileCursor cur(a);
  int panel = cur.tn;
  const int ashift = a.n_abuf - 1;                          // n_abuf is 1 or 2
  const uint32_t a_img_bytes = (uint32_t)a.atoms * WT2_ATOM_BYTES;
  const int atoms = R > 0 ? (2 * R + 31) / 32 : a.atoms;
  int acc = 0; uint32_t acc_phase = 0;
  int slot = 0; uint32_t slot_phase = 0;
  int pseq = 0, ab = 0;
  if (!bounded_wait(&bars->afull[0], 0u, bars)) return;
  for (; cur.valid();) {
    if (!bounded_wait(&bars->tmem_empty[acc], acc_phase ^ 1, bars)) return;
    ptx::tc_fence_after_sync();
    const uint32_t d_tmem = tmem_base + (uint32_t)(acc * WT2_COLS);
    const uint32_t acat_a = acat_addr + (uint32_t)ab * a_img_bytes;
#pragma unroll
    for (int c = 0; c < (R > 0 ? atoms : WT2_MAX_ATOMS); ++c) {
      if (R == 0 && c >= atoms) break;
      if (!bounded_wait(&bars->bfull[slot], slot_phase, bars)) return;
      ptx::tc_fence_after_sync();
      issue_chunk_mmas<R>(c, a.p.rank, bslot_addr + (uint32_t)slot * WT2_ATOM_BYTES, acat_a, d_tmem);
      ptx::mma_commit(&bars->bempty[slot]);        // the chunk may be overwritten once these MMAs have read it
      if (++slot == a.n_bslot) { slot = 0; slot_phase ^= 1; }
    }
    ptx::mma_commit(&bars->tmem_full[acc]);
    if (++acc == WT2_ACC) { acc = 0; acc_phase ^= 1; }
    cur.next();
    if (cur.valid() && cur.tn != panel) {
      // the MMAs issued so far are the last readers of this panel's A image; the next panel's is in the other
      // buffer (or about to replace this one)
      ptx::mma_commit(&bars->aempty[ab]);
      panel = cur.tn;
      ++pseq;
      ab = pseq & ashift;
      if (!bounded_wait(&bars->afull[ab], (uint32_t)((pseq >> ashift) & 1), bars)) return;
    }
  }
}

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
  uint8_t* acat_base = out_base + (size_t)a.n_out * a.out_bytes;        // A image buffer b: atoms x 16 KB
  const uint32_t a_img_bytes = (uint32_t)a.atoms * WT2_ATOM_BYTES;
  uint8_t* bslot_base = acat_base + (size_t)a.n_abuf * a_img_bytes;     // ring of 16 KB chunks of B images
  float* sb_base = reinterpret_cast<float*>(bslot_base + (size_t)a.n_bslot * WT2_ATOM_BYTES);
  WtileBarriers* bars = reinterpret_cast<WtileBarriers*>(reinterpret_cast<uint8_t*>(sb_base) + wtile_sb_region_bytes(a));
  const Params& p = a.p;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr bool HAS_OUT1 = (MODE == WT2_PACK);      // staged in shared memory: the code words of the export
  constexpr bool READ_ONLY = !wt2_has_wq(MODE);      // W0 stages are read, never written back

  if (threadIdx.x == 0) {
    const uint32_t op_arrivals = a.op_img ? 1 : WT2_BUILDERS;   // one thread announcing a bulk copy, or the builders of the atom
    for (int i = 0; i < WT2_MAX_STAGES; ++i) {
      ptx::mbar_init(&bars->full[i], 1);
      // the export does not write back into the stage: the group that read it hands it back itself
      ptx::mbar_init(&bars->empty[i], READ_ONLY ? WT2_GROUP_THREADS : 1);
      ptx::mbar_init(&bars->written[i], WT2_GROUP_THREADS);
    }
    for (int i = 0; i < WT2_GROUPS; ++i) ptx::mbar_init(&bars->out_empty[i], 1);
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&bars->afull[i], op_arrivals);
      ptx::mbar_init(&bars->aempty[i], 1);
    }
    for (int i = 0; i < WT2_MAX_BSLOTS; ++i) {
      ptx::mbar_init(&bars->bfull[i], op_arrivals);
      ptx::mbar_init(&bars->bempty[i], 1);
    }
    for (int i = 0; i < WT2_ACC; ++i) {
      ptx::mbar_init(&bars->tmem_full[i], 1);
      ptx::mbar_init(&bars->tmem_empty[i], WT2_GROUP_THREADS);
    }
    bars->abort = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tmap_w0);
    ptx::prefetch_tmap(&tmap_out0);
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

  if (warp >= WT2_FIRST_EPI_WARP && warp < WT2_SECOND_STORE_WARP) {
    // the epilogue warps have nothing to do until the first merge is complete: they clear the caller's buffers
    const size_t stride = (size_t)gridDim.x * WT2_EPI_THREADS;
    const size_t first = (size_t)blockIdx.x * WT2_EPI_THREADS + (threadIdx.x - WT2_FIRST_EPI_WARP * 32);
#pragma unroll
    for (int z = 0; z < 4; ++z)
      for (size_t e = first; e < a.zero.n[z]; e += stride) a.zero.ptr[z][e] = 0.f;
  }

  if (warp == 0) {
    // ------------------------------ TMA loads of W0 ---------------------------
    if (lane == 0) {
      StageSeq seq0(0, a.n_stages), seq1(1, a.n_stages);
      static_assert(WT2_GROUPS == 2, "one stage sequence per epilogue group");
      int grp = 0;                                   // tile i belongs to group i % WT2_GROUPS
      for (TileCursor cur(a); !bars->abort && cur.valid(); cur.next()) {
        const int m0 = cur.m0(), n0 = cur.n0();
        StageSeq& sq = grp ? seq1 : seq0;
        const int stage = sq.stage();
        if (!bounded_wait(&bars->empty[stage], sq.parity() ^ 1, bars)) break;
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
        sq.advance();
        grp ^= 1;
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------ merge MMAs --------------------------------
    if (lane == 0) {
      switch (p.rank) {
        case 8: wtile_mma_role<8>(a, bars, tmem_base, ptx::smem_u32(acat_base), ptx::smem_u32(bslot_base)); break;
        case 16: wtile_mma_role<16>(a, bars, tmem_base, ptx::smem_u32(acat_base), ptx::smem_u32(bslot_base)); break;
        case 32: wtile_mma_role<32>(a, bars, tmem_base, ptx::smem_u32(acat_base), ptx::smem_u32(bslot_base)); break;
        case 64: wtile_mma_role<64>(a, bars, tmem_base, ptx::smem_u32(acat_base), ptx::smem_u32(bslot_base)); break;
        default: wtile_mma_role<0>(a, bars, tmem_base, ptx::smem_u32(acat_base), ptx::smem_u32(bslot_base)); break;
      }
    }
    __syncwarp();
  } else if (warp == 2 || warp == WT2_SECOND_STORE_WARP) {
    // ------------------------------ TMA stores --------------------------------
    // Two issuing threads, one per epilogue group (tiles sid, sid + 2, ...): a thread hands a stage back only
    // after its copy has read it, which takes the TMA unit a thousand cycles or more behind the loads queued
    // before it, and one thread doing that for every tile in turn was the slowest role of the kernel.
    if (lane == 0 && (wt2_has_wq(MODE) || MODE == WT2_PACK)) {
      const int sid = warp == 2 ? 0 : 1;
      StageSeq sq(sid, a.n_stages);
      const int ob = sid;                            // the group's own staging buffer of code words
      for (TileCursor cur(a, sid, WT2_GROUPS); !bars->abort && cur.valid(); cur.next()) {
        const int m0 = cur.m0(), n0 = cur.n0();
        const int stage = sq.stage();
        if (!bounded_wait(&bars->written[stage], sq.parity(), bars)) break;
        const uint8_t* src = stage_base + (size_t)stage * WT2_STAGE_BYTES;
        const uint8_t* src1 = out_base + (size_t)ob * a.out_bytes;
        const bool second_box = n0 + 64 < p.d_in;
        if constexpr (!READ_ONLY) {
          ptx::tma_store_2d(&tmap_out0, src, n0, m0);
          if (second_box) ptx::tma_store_2d(&tmap_out0, src + WT2_STAGE_BYTES / 2, n0 + 64, m0);
        }
        if constexpr (MODE == WT2_PACK) ptx::tma_store_2d(&tmap_out0, src1, (n0 * p.bits) >> 5, m0);
        ptx::bulk_commit_group();
        // hand the buffers back as soon as the copies have read them: a stage that is released a tile later is a
        // load that starts a tile later
        ptx::bulk_wait_group_read0();
        if constexpr (!READ_ONLY) ptx::mbar_arrive(&bars->empty[stage]);
        if constexpr (HAS_OUT1) ptx::mbar_arrive(&bars->out_empty[ob]);
        sq.advance();
      }
      ptx::bulk_wait_group0();
    }
    __syncwarp();
  } else if (warp == 3) {
    // ------------------------------ MMA operands ------------------------------
    // With ready-made images one thread issues bulk copies; without, the warp builds each atom from A and B.
    const bool img = a.op_img != nullptr;
    const int btid = lane;                           // builder thread index
    if (img ? btid == 0 : true) {
      if (img) ptx::griddep_wait();                  // k_split_operands has written the images
      int slot = 0; uint32_t slot_phase = 0;
      int panel = -1, pseq = -1;
      const int ashift = a.n_abuf - 1;
      for (TileCursor cur(a); !bars->abort && cur.valid(); cur.next()) {
        if (cur.tn != panel) {
          panel = cur.tn; ++pseq;
          const int ab = pseq & ashift, use = pseq >> ashift;     // earlier fills of this buffer
          if (use >= 1) bounded_wait(&bars->aempty[ab], (uint32_t)((use - 1) & 1), bars);
          if (bars->abort) break;
          uint8_t* acat = acat_base + (size_t)ab * a_img_bytes;
          if (img) {
            ptx::mbar_arrive_expect_tx(&bars->afull[ab], a_img_bytes);
            ptx::bulk_load(acat, a.op_img + (size_t)cur.tn * a_img_bytes, a_img_bytes, &bars->afull[ab]);
          } else {
            for (int c = 0; c < a.atoms; ++c) build_atom_a<WT2_BUILDERS>(a, cur.n0(), c, acat + (size_t)c * WT2_ATOM_BYTES, btid);
            ptx::fence_proxy_async_smem();
            ptx::mbar_arrive(&bars->afull[ab]);
          }
        }
        for (int c = 0; c < a.atoms; ++c) {
          bounded_wait(&bars->bempty[slot], slot_phase ^ 1, bars);
          if (bars->abort) break;
          uint8_t* chunk = bslot_base + (size_t)slot * WT2_ATOM_BYTES;
          if (img) {
            ptx::mbar_arrive_expect_tx(&bars->bfull[slot], WT2_ATOM_BYTES);
            ptx::bulk_load(chunk, a.op_img + ((size_t)(a.tiles_n + cur.tm) * a.atoms + c) * WT2_ATOM_BYTES,
                           WT2_ATOM_BYTES, &bars->bfull[slot]);
          } else {
            build_atom_b<WT2_BUILDERS>(a, cur.m0(), c, chunk, btid);
            ptx::fence_proxy_async_smem();
            ptx::mbar_arrive(&bars->bfull[slot]);
          }
          if (++slot == a.n_bslot) { slot = 0; slot_phase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp >= WT2_FIRST_EPI_WARP && warp < WT2_SECOND_STORE_WARP) {
    // ------------------------------ epilogue ----------------------------------
    // Two groups of eight warps; group grp owns the CTA's tiles i = grp, grp + 2, ... (accumulator stage i % 4).
    // A thread is one weight row (TMEM lane) and one 64-column half of its group's tile.  The groups meet only
    // through the mbarriers: while one waits for a merge or a tile, the other keeps the pipes busy.  (Three groups
    // were measured: each tile then takes longer, the stages are held longer, and nothing is gained.)
    const int quarter = warp & 3;
    const int grp = (warp - WT2_FIRST_EPI_WARP) >> 3;
    const int chalf = ((warp - WT2_FIRST_EPI_WARP) >> 2) & 1;   // column half of the tile
    const int row = quarter * 32 + lane;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const int sbw = 2 * a.ngt;                                  // floats per thread: s x ngt | b x ngt
    float* grp_sb = sb_base + (size_t)grp * 2 * WT2_ROWS * sbw;   // two buffers of [128 rows][s x ngt | b x ngt]
    const bool stage_sb_self = !a.fast && !a.sb_box;            // the group copies s and b itself

    // ---- s and b of the tile's rows for the quantization groups it intersects: the threads of column half 0
    //      (one per weight row) copy them with asynchronous 4-byte copies into the group's buffer for its next
    //      tile; the group meets at a named barrier when it starts that tile.  (Each row's values sit in a line
    //      of their own, so every copy instruction touches 32 lines: the fewer of them the better.) ----
    auto stage_sb = [&](int m0_, int n0_, int buf) {
      if (chalf != 0 || !stage_sb_self) return;
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
    // ---- fast path: s and b of this thread's half row of an interior tile, straight from global memory ----
    auto interior = [&](int m0_, int n0_) { return a.fast && m0_ + WT2_ROWS <= p.d_out && n0_ + WT2_COLS <= p.d_in; };
    auto fetch_sb = [&](int m0_, int n0_, float& s_out, float& b_out) {
      if (!interior(m0_, n0_)) return;
      const size_t idx = (size_t)(m0_ + row) * p.ngroups + group_of(a, n0_ + chalf * 64);
      s_out = __ldg(a.s + idx); b_out = __ldg(a.b + idx);
    };

    TileCursor cur(a, grp, WT2_GROUPS);
    float s_next = 1.f, b_next = 0.f;
    if (cur.valid()) {
      stage_sb(cur.m0(), cur.n0(), 0);
      fetch_sb(cur.m0(), cur.n0(), s_next, b_next);
    }
    int sb_buf = 0;
    const int qn_bits = kRoundMagicBits + (int)p.qn;
    [[maybe_unused]] float e_quant = 0.f, e_clip = 0.f;         // WT2_ERROR: this thread's partial sums

    // the group's own W0 stages and staging buffer of code words (no division per tile: that is dozens of
    // instructions, on warps whose issue slots are the scarce thing here)
    StageSeq sq(grp, a.n_stages);
    const int ob = grp;
    [[maybe_unused]] int ob_uses = 0;
    for (int i = grp; cur.valid(); cur.next(), i += WT2_GROUPS) {
      const int stage = sq.stage();
      const uint32_t phase = sq.parity();
      const int m0 = cur.m0(), n0 = cur.n0();
      const int o = m0 + row;
      const bool row_ok = o < p.d_out;
      const int acc = i & 3;
      const int g_first = group_of(a, n0);
      int m1 = 0, n1 = 0;
      const bool has_next = cur.peek(1, m1, n1);
      const float s_cur = s_next, b_cur = b_next;
      if (has_next) fetch_sb(m1, n1, s_next, b_next);           // in flight while this tile is worked on
      const float *my_s, *my_b;                                 // s and b of this row, from group sb_first on
      int sb_first;
      if (a.fast) {                                             // general tiles of a fast launch (edges): global memory
        my_s = a.s + (size_t)o * p.ngroups;
        my_b = a.b + (size_t)o * p.ngroups;
        sb_first = 0;
      } else if (a.sb_box) {                                    // they arrive with the W0 tile (full[stage] below)
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
      bounded_wait(&bars->full[stage], phase, bars);
      if constexpr (HAS_OUT1) {
        if (ob_uses >= 1) bounded_wait(&bars->out_empty[ob], (uint32_t)((ob_uses - 1) & 1), bars);
      }
      uint8_t* tile_rows = stage_base + (size_t)stage * WT2_STAGE_BYTES + row * 128;
      // second output: the export's staging rows in shared memory; the STE factors go straight to the tile's block
      // of the factor array in global memory (16 bytes per thread and piece, a warp's 32 rows contiguous)
      [[maybe_unused]] uint8_t* out1 =
          wt2_has_factors(MODE)
              ? reinterpret_cast<uint8_t*>(a.F + ((size_t)cur.tm * a.tiles_n + cur.tn) * FACTOR_TILE_ELEMS)
              : out_base + (size_t)ob * a.out_bytes;
      if (interior(m0, n0)) {
        // the thread's 64 columns lie in one quantization group
        FastConsts fc;
        fc.s = s_cur; fc.b = b_cur; fc.rs = 1.0f / s_cur;
        fc.qn = p.qn; fc.qp = p.qp; fc.gamma = p.gamma;
        const uint32_t taddr = tmem_base + lane_base + (uint32_t)(acc * WT2_COLS + chalf * 64);
        if constexpr (MODE == WT2_PACK) {
          if (p.bits == 4) wtile_half_row_fast<MODE, 4>(fc, taddr, tile_rows, row, chalf, out1, &bars->tmem_empty[acc], e_quant, e_clip);
          else wtile_half_row_fast<MODE, 3>(fc, taddr, tile_rows, row, chalf, out1, &bars->tmem_empty[acc], e_quant, e_clip);
          const int g = group_of(a, n0 + chalf * 64);
          if ((n0 + chalf * 64) - g * p.group == 0) {             // first half row of its group
            a.s16[(size_t)o * p.ngroups + g] = __float2half_rn(fc.s);
            a.b16[(size_t)o * p.ngroups + g] = __float2half_rn(fc.b);   // Q_N = 0: b + s Q_N = b
          }
        } else {
          wtile_half_row_fast<MODE, 4>(fc, taddr, tile_rows, row, chalf, out1, &bars->tmem_empty[acc], e_quant, e_clip);
        }
      } else {
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
              if constexpr (MODE == WT2_ERROR) {
                if (ok) {                                                           // |W_comb - W_q|, and its part outside the range
                  const float2 t2 = __fadd2_rn(w, make_float2(-wcl.x, -wcl.y));
                  const float ex = fabsf(wc.x - q.x), ey = fabsf(wc.y - q.y);
                  e_quant += ex + ey;
                  e_clip += (fabsf(t2.x) > kMaskGuard ? ex : 0.f) + (fabsf(t2.y) > kMaskGuard ? ey : 0.f);
                }
              }
              if constexpr (wt2_has_factors(MODE)) {
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
            if constexpr (wt2_has_wq(MODE)) {
              uint4 o4;
              o4.x = pack_bf16x2(wq[0], wq[1]); o4.y = pack_bf16x2(wq[2], wq[3]);
              o4.z = pack_bf16x2(wq[4], wq[5]); o4.w = pack_bf16x2(wq[6], wq[7]);
              *reinterpret_cast<uint4*>(tile_rows + chunk) = o4;                    // in place, same swizzled position
            }
            if constexpr (wt2_has_factors(MODE)) {
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
      }
      ptx::fence_proxy_async_smem();                   // the stores above are read by TMA
      ptx::mbar_arrive(&bars->written[stage]);
      if constexpr (READ_ONLY) ptx::mbar_arrive(&bars->empty[stage]);   // W0 has been read
      sb_buf ^= 1;
      if (has_next) stage_sb(m1, n1, sb_buf);          // the other buffer: its readers passed this tile's barrier
      sq.advance();
      ++ob_uses;
    }
    if constexpr (MODE == WT2_ERROR) {                 // the warp's partial sums, then one fp64 atomic per warp and sum
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        e_quant += __shfl_xor_sync(0xffffffffu, e_quant, off);
        e_clip += __shfl_xor_sync(0xffffffffu, e_clip, off);
      }
      if (lane == 0) {
        atomicAdd(a.errors, (double)e_quant);
        atomicAdd(a.errors + 1, (double)e_clip);
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
// The operands of the merge take one or two A-image buffers and a ring of 16 KB chunks of B images.  Of the
// combinations that fit, the best by this order of concerns is taken: at least 3 stages; two staging buffers;
// a ring that holds more than one tile's chunks; at least 4 stages; two A buffers; a ring of two tiles; 5 stages.
// `sb_by_tma`: s and b may come in by TMA (the caller has checked their alignment); the shape must allow it too.
inline bool wtile_plan(WtileArgs& a, int mode, bool sb_by_tma = true) {
  const Params& p = a.p;
  a.atoms = (2 * p.rank + 31) / 32;
  a.ngt = std::min(p.ngroups, (WT2_COLS - 1) / p.group + 2);
  a.group_shift = -1;
  for (int sh = 3; sh < 31; ++sh)
    if ((1 << sh) == p.group) a.group_shift = sh;
  // (the export's fast path builds its code words from the raw rounding results, which it does for the unsigned grid)
  a.fast = (p.group % 64 == 0 && (mode != WT2_PACK || (p.qn == 0.f && (p.bits == 3 || p.bits == 4)))) ? 1 : 0;   // (WT2_ERROR: as the dequantize modes)
  // a box starts at a group column that is a multiple of 4 (16 bytes) at or below the tile's first group, so it
  // is up to 3 groups wider than the tile; the row pitch of s and b must be a multiple of 16 bytes
  const int box = (a.ngt + 3 + 3) / 4 * 4;
  a.sb_box = (!a.fast && sb_by_tma && p.ngroups % 4 == 0 && p.ngroups >= box && box <= 256) ? box : 0;
  a.out_bytes = mode == WT2_PACK ? WT2_ROWS * (WT2_COLS * p.bits / 8) : 0;
  const bool has_out = mode == WT2_PACK;
  long best = -1;
  WtileArgs pick = a;
  const int ring_opts[4] = {2 * a.atoms, a.atoms + 1, 3, 2};
  for (int stages = 2; stages <= WT2_MAX_STAGES; ++stages)
    for (int n_out = has_out ? WT2_GROUPS : 0; n_out <= (has_out ? WT2_GROUPS : 0); ++n_out)   // one per group
      for (int n_abuf = 1; n_abuf <= 2; ++n_abuf)
        for (int ro = 0; ro < 4; ++ro) {
          const int ring = ring_opts[ro];
          if (ring < 2 || ring > WT2_MAX_BSLOTS) continue;
          WtileArgs c = a;
          c.n_stages = stages; c.n_out = n_out; c.n_abuf = n_abuf; c.n_bslot = ring;
          if (wtile_smem_bytes(c) > 227 * 1024) continue;
          long score = 0;
          score = score * 2 + (stages >= 3);
          score = score * 2 + (!has_out || n_out >= 2);
          score = score * 2 + (ring > a.atoms);
          score = score * 2 + (stages >= 4);
          score = score * 2 + (n_abuf == 2);
          score = score * 2 + (ring >= 2 * a.atoms);
          score = score * 2 + (stages >= 5);
          score = score * 2 + (!has_out || n_out >= WT2_GROUPS);
          score = score * 16 + ring;                 // then the deeper ring
          if (score > best) { best = score; pick = c; }
        }
  if (best < 0) return false;
  a = pick;
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
  return wtile_plan(a, mode);                       // the shared-memory plan must fit
}

// mode WT2_DEQUANT: out0 = W_q.  WT2_DEQUANT_F: out0 = W_q, out1 = STE factors.  WT2_PACK: out0 = codes.
// WT2_ERROR: no outputs but `errors` (two doubles, zero on entry).
// Bytes of the operand images of a problem (see k_split_operands).
inline size_t wtile_image_bytes(const Params& p) {
  const size_t atoms = (2 * (size_t)p.rank + 31) / 32;
  return ((size_t)ceil_div(p.d_out, WT2_ROWS) + (size_t)ceil_div(p.d_in, WT2_COLS)) * atoms * WT2_ATOM_BYTES;
}

// `copies` (optional, needs `op_img`): the operand-split launch also writes these bf16 copies of A and B^T.
// `op_img` (optional, wtile_image_bytes(p) bytes of device scratch, 16-byte aligned): with it the MMA operands are
// split once by a launch of k_split_operands and reach the tiles by bulk copies; without it one warp of every CTA
// builds them tile by tile (slower).  `zero` (optional): buffers that launch also clears; *zeroed is set when it did.
inline l4q_status launch_wtile_tc(int mode, const Params& p, const void* W0, const float* A, const float* B,
                                  const float* s, const float* b, void* out0, void* out1, __half* s16, __half* b16,
                                  cudaStream_t st, void* op_img = nullptr, const ZeroList* zero = nullptr,
                                  bool* zeroed = nullptr, const Bf16Copies* copies = nullptr, double* errors = nullptr) {
  WtileArgs a{};
  a.p = p; a.A = A; a.B = B; a.s = s; a.b = b; a.s16 = s16; a.b16 = b16; a.errors = errors;
  a.tiles_m = ceil_div(p.d_out, WT2_ROWS);
  a.tiles_n = ceil_div(p.d_in, WT2_COLS);
  const bool sb_aligned = ((reinterpret_cast<uintptr_t>(s) | reinterpret_cast<uintptr_t>(b)) & 15u) == 0;
  if (!wtile_plan(a, mode, sb_aligned)) return L4Q_ERR_UNSUPPORTED;
  CUtensorMap t_w0, t_o0, t_o1, t_s, t_b;
  if (!make_tmap_bf16(&t_w0, W0, p.d_out, p.d_in, WT2_ROWS)) return cuda_fail();
  t_o1 = t_w0;
  if (mode == WT2_PACK) {
    if (!make_tmap_words(&t_o0, out0, p.d_out, ((uint64_t)p.d_in * p.bits) >> 5, WT2_COLS * p.bits / 32))
      return cuda_fail();
  } else if (mode == WT2_ERROR || mode == WT2_FACTORS) {
    t_o0 = t_w0;                                    // nothing is stored by TMA
    a.F = reinterpret_cast<__half*>(out1);
  } else {
    if (!make_tmap_bf16(&t_o0, out0, p.d_out, p.d_in, WT2_ROWS)) return cuda_fail();
    a.F = reinterpret_cast<__half*>(out1);
  }
  t_s = t_w0; t_b = t_w0;                          // placeholders when unused
  if (a.sb_box) {                                   // fp32 moved as 32-bit words
    if (!make_tmap_words(&t_s, s, p.d_out, p.ngroups, a.sb_box) || !make_tmap_words(&t_b, b, p.d_out, p.ngroups, a.sb_box))
      return cuda_fail();
  }
  const int grid = std::min(a.tiles_m * a.tiles_n, sm_count());
#ifdef L4Q_EXPERIMENT
  if (const char* e = getenv("L4Q_WT_STAGES")) a.n_stages = std::min(a.n_stages, atoi(e));
  if (const char* e = getenv("L4Q_WT_OPS")) {     // "abuf,ring,stages"
    int x = 0, y = 0, z = 0;
    if (sscanf(e, "%d,%d,%d", &x, &y, &z) == 3) {
      WtileArgs c = a; c.n_abuf = x; c.n_bslot = y; c.n_stages = z;
      if (wtile_smem_bytes(c) <= 227 * 1024) a = c;
    }
  }
#endif
  const size_t smem = wtile_smem_bytes(a);
#ifdef L4Q_EXPERIMENT
  if (const char* e = getenv("L4Q_WT_IMG")) { if (!atoi(e)) op_img = nullptr; }
#endif
  if (op_img) {
    const int image_blocks = (a.tiles_n + a.tiles_m) * a.atoms * 4;
    Bf16Copies cp{};
    int copy_blocks = 0;
    if (copies) {
      cp = *copies;
      copy_blocks = (int)(((long long)cp.rn * (p.d_in + p.d_out) / 8 + 255) / 256);
    }
    k_split_operands<<<image_blocks + copy_blocks, 256, 0, st>>>(a, static_cast<uint8_t*>(op_img), image_blocks, cp);
    if (cudaGetLastError() != cudaSuccess) return cuda_fail();
    a.op_img = static_cast<const uint8_t*>(op_img);
  }
  if (zero) {                                       // the kernel's epilogue warps clear these before their first tile
    a.zero = *zero;
    if (zeroed) *zeroed = true;
  }
  auto launch = [&](auto kern) -> l4q_status {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return cuda_fail();
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(WT2_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = op_img ? 1 : 0;                  // overlap with the operand split that was just launched
    if (cudaLaunchKernelEx(&cfg, kern, t_w0, t_o0, t_o1, t_s, t_b, a) != cudaSuccess) {
      cudaGetLastError();
      return cuda_fail();
    }
    return cudaGetLastError() == cudaSuccess ? L4Q_OK : L4Q_ERR_CUDA;
  };
  switch (mode) {
    case WT2_DEQUANT: return launch(k_wtile_tc<WT2_DEQUANT>);
    case WT2_DEQUANT_F: return launch(k_wtile_tc<WT2_DEQUANT_F>);
    case WT2_ERROR: return launch(k_wtile_tc<WT2_ERROR>);
    case WT2_FACTORS: return launch(k_wtile_tc<WT2_FACTORS>);
    default: return launch(k_wtile_tc<WT2_PACK>);
  }
}

}  // namespace l4q
