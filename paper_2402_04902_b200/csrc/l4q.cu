// C ABI of the L4Q library (see include/l4q.h): argument validation, workspace
// layout and kernel launches.  One translation unit; the kernels live in the
// headers included below.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <vector>

#include "l4q_common.cuh"
#include "l4q_quant.cuh"
#include "l4q_val.cuh"
#include "l4q_gemm.cuh"
#include "l4q_wtile.cuh"
#include "l4q_init.cuh"
#include "l4q_infer.cuh"
#include "l4q_variants.cuh"
#include "l4q_tilecopy.cuh"

using namespace l4q;

namespace {

std::atomic<uint64_t> g_launches{0};

// ---- optional per-kernel timing (l4q_profile_*) ------------------------------
struct ProfSlot { cudaEvent_t begin, end; int kernel; };
std::mutex g_prof_mu;
bool g_prof_on = false;
std::vector<ProfSlot> g_prof_pool;
size_t g_prof_used = 0;
double g_prof_ms[L4Q_KERNEL_COUNT];
uint64_t g_prof_n[L4Q_KERNEL_COUNT];
constexpr size_t kProfPool = 8192;

// Brackets one kernel launch: counts it and, when profiling is on, records a pair of events around it.
class KernelScope {
 public:
  KernelScope(int kernel, cudaStream_t st) : st_(st) {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    std::lock_guard<std::mutex> lk(g_prof_mu);
    if (g_prof_on && g_prof_used < g_prof_pool.size()) {
      slot_ = (long)g_prof_used++;
      g_prof_pool[slot_].kernel = kernel;
      cudaEventRecord(g_prof_pool[slot_].begin, st_);
    }
  }
  ~KernelScope() {
    if (slot_ >= 0) cudaEventRecord(g_prof_pool[slot_].end, st_);
  }
 private:
  cudaStream_t st_;
  long slot_ = -1;
};

void prof_drain_locked() {
  for (size_t i = 0; i < g_prof_used; ++i) {
    float ms = 0.f;
    if (cudaEventSynchronize(g_prof_pool[i].end) == cudaSuccess &&
        cudaEventElapsedTime(&ms, g_prof_pool[i].begin, g_prof_pool[i].end) == cudaSuccess) {
      g_prof_ms[g_prof_pool[i].kernel] += ms;
      g_prof_n[g_prof_pool[i].kernel] += 1;
    }
  }
  g_prof_used = 0;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Checks of the problem statement common to all ops.  Fills the kernel parameters.
l4q_status make_params(const l4q_desc* d, Params* p) {
  if (!d) return L4Q_ERR_INVALID_ARG;
  if (d->tokens <= 0 || d->d_in <= 0 || d->d_out <= 0 || d->rank <= 0 || d->group_size <= 0)
    return L4Q_ERR_INVALID_ARG;
  if (d->io_dtype != L4Q_BF16 && d->io_dtype != L4Q_F32) return L4Q_ERR_INVALID_ARG;
  if (!(d->alpha == d->alpha) || !(d->grad_scale == d->grad_scale)) return L4Q_ERR_INVALID_ARG;
  if (d->tokens > (1 << 30) || d->d_in > (1 << 30) || d->d_out > (1 << 30)) return L4Q_ERR_UNSUPPORTED;
  if (d->bits < 2 || d->bits > 8) return L4Q_ERR_UNSUPPORTED;
  if (d->d_in % d->group_size != 0) return L4Q_ERR_UNSUPPORTED;
  if (d->group_size % 8 != 0 || d->d_in % 8 != 0) return L4Q_ERR_UNSUPPORTED;
  if (d->rank > L4Q_MAX_RANK) return L4Q_ERR_UNSUPPORTED;   // the plain-ALU weight-tile kernel keeps rank x 320 floats in shared memory
  if (d->io_dtype == L4Q_BF16 && d->d_out % 8 != 0) return L4Q_ERR_UNSUPPORTED;
  p->tokens = (int)d->tokens; p->d_in = (int)d->d_in; p->d_out = (int)d->d_out;
  p->rank = d->rank; p->bits = d->bits; p->group = d->group_size;
  p->ngroups = (int)(d->d_in / d->group_size);
  p->gamma = d->alpha / (float)d->rank;
  if (d->flags & L4Q_FLAG_SIGNED_GRID) {
    p->qn = -(float)(1 << (d->bits - 1)); p->qp = (float)((1 << (d->bits - 1)) - 1);
  } else {
    p->qn = 0.f; p->qp = (float)((1 << d->bits) - 1);
  }
  p->grad_scale = d->grad_scale;
  return L4Q_OK;
}

// The bf16 weight-gradient epilogue is instantiated for these ranks only.
bool wgrad_rank_supported(int rank) { return rank == 8 || rank == 16 || rank == 32 || rank == 64; }

size_t wq_scratch_bytes(const l4q_desc* d) {
  const size_t esz = d->io_dtype == L4Q_BF16 ? 2 : 4;
  return align_up((size_t)d->d_out * (size_t)d->d_in * esz, 256);
}

// Scratch of the split LoRA operands of the tensor-core weight-tile kernel (bf16 mode).
size_t operand_image_bytes(const l4q_desc* d, const Params& p) {
  return d->io_dtype == L4Q_BF16 && wtile_tc_supported(p, WT2_DEQUANT) ? align_up(wtile_image_bytes(p), 256) : 0;
}

// bf16 copies of A and B^T for the weight-gradient kernel (rows up to the MMA's N, see Bf16Copies)
size_t wgrad_copy_bytes(const l4q_desc* d, const Params& p) {
  if (d->io_dtype != L4Q_BF16 || !wgrad_rank_supported(p.rank)) return 0;
  const size_t rn = (size_t)wgrad_rn(p.rank);
  return align_up(rn * p.d_in * 2, 256) + align_up(rn * p.d_out * 2, 256);
}

size_t factor_scratch_bytes(const l4q_desc* d) {
  return align_up(factor_elems((int)d->d_out, (int)d->d_in) * sizeof(__half), 256);
}

inline l4q_status launch_status() { return cudaGetLastError() == cudaSuccess ? L4Q_OK : L4Q_ERR_CUDA; }

// The bf16 copies of A and B^T inside a scratch region of wgrad_copy_bytes().
Bf16Copies carve_copies(const Params& p, void* base) {
  Bf16Copies cp{};
  cp.rn = wgrad_rn(p.rank);
  cp.A16 = reinterpret_cast<__nv_bfloat16*>(base);
  cp.Bt16 = reinterpret_cast<__nv_bfloat16*>(static_cast<unsigned char*>(base) + align_up((size_t)cp.rn * p.d_in * 2, 256));
  return cp;
}

// The copies by a launch of their own (where no operand-split launch made them).
l4q_status launch_copies(const Params& p, const float* A, const float* B, const Bf16Copies& cp, cudaStream_t st) {
  WtileArgs a{};
  a.p = p; a.A = A; a.B = B;
  const int blocks = (int)(((long long)cp.rn * (p.d_in + p.d_out) / 8 + 255) / 256);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  k_split_operands<<<blocks, 256, 0, st>>>(a, nullptr, 0, cp);
  return launch_status();
}

// Merge + fake-quantize the whole weight into `wq` (io dtype) -- the recompute step of fwd and bwd.
// `fac` (optional, bf16 mode only) also receives the fp16 STE factors the weight-gradient kernel reads.
template <bool IO_BF16>
l4q_status launch_dequant(const Params& p, const void* W0, const float* A, const float* B, const float* s,
                          const float* b, void* wq, __half* fac, cudaStream_t st, void* op_img = nullptr,
                          const ZeroList* zero = nullptr, bool* zeroed = nullptr, const Bf16Copies* copies = nullptr,
                          bool* copied = nullptr) {
  if constexpr (IO_BF16) {
    const int mode = fac ? (wq ? WT2_DEQUANT_F : WT2_FACTORS) : WT2_DEQUANT;
    if (wtile_tc_supported(p, mode)) {               // tensor-core merge, TMA in and out
      KernelScope ks(L4Q_KERNEL_DEQUANT, st);   // covers the operand split too, which is one more launch
      if (op_img) g_launches.fetch_add(1, std::memory_order_relaxed);
      if (op_img && copies && copied) *copied = true;
      return launch_wtile_tc(mode, p, W0, A, B, s, b, wq, fac, nullptr, nullptr, st, op_img, zero, zeroed,
                             op_img ? copies : nullptr);
    }
  }
  const size_t smem = weight_tile_smem_bytes(p.rank);
  auto kern = k_weight_tile<IO_BF16, WT_MODE_DEQUANT>;
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return cuda_fail();
  dim3 grid(ceil_div(p.d_in, WT_COLS), ceil_div(p.d_out, WT_ROWS));
  KernelScope ks(L4Q_KERNEL_DEQUANT, st);
  kern<<<grid, WT_THREADS, smem, st>>>(p, W0, A, B, s, b, wq, fac, nullptr, nullptr, nullptr, nullptr);
  return launch_status();
}

template <bool IO_BF16>
l4q_status launch_pack(const Params& p, const void* W0, const float* A, const float* B, const float* s,
                       const float* b, uint32_t* codes, __half* s16, __half* b16, cudaStream_t st,
                       void* op_img = nullptr) {
  if constexpr (IO_BF16) {
    if (wtile_tc_supported(p, WT2_PACK)) {
      KernelScope ks(L4Q_KERNEL_PACK, st);      // covers the operand split too, which is one more launch
      if (op_img) g_launches.fetch_add(1, std::memory_order_relaxed);
      return launch_wtile_tc(WT2_PACK, p, W0, A, B, s, b, codes, nullptr, s16, b16, st, op_img);
    }
  }
  const size_t smem = weight_tile_smem_bytes(p.rank);
  auto kern = k_weight_tile<IO_BF16, WT_MODE_PACK>;
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return cuda_fail();
  dim3 grid(ceil_div(p.d_in, WT_COLS), ceil_div(p.d_out, WT_ROWS));
  KernelScope ks(L4Q_KERNEL_PACK, st);
  kern<<<grid, WT_THREADS, smem, st>>>(p, W0, A, B, s, b, nullptr, nullptr, codes, s16, b16, nullptr);
  return launch_status();
}

// ---- LoRA and QAT-LoRA layers (Eq. 1-2, Sec. 3.1) ---------------------------------------------

struct LoraWorkspace {
  void* wq = nullptr;            // QAT-LoRA: Q(W0), bf16
  __half* fac = nullptr;         // QAT-LoRA backward: STE factors
  VariantScratch v{};
  float* zero_B = nullptr;       // QAT-LoRA: a zero LoRA factor, so that the weight-tile kernel quantizes W0 alone
  void* op_img = nullptr;        // QAT-LoRA: the split operands of that kernel's merge (operand_image_bytes)
  float *dA_unused = nullptr, *dB_unused = nullptr;   // QAT-LoRA backward: the merged-layer LoRA gradients, not wanted
  void* copies = nullptr;        // QAT-LoRA backward: bf16 copies of A and the zero factor for the weight-gradient kernel
  size_t bytes = 0;
};

LoraWorkspace lora_workspace(const l4q_desc* d, const Params& p, int kind, int op, void* base) {
  LoraWorkspace w;
  unsigned char* c = static_cast<unsigned char*>(base);
  size_t off = 0;
  auto take = [&](size_t n) { unsigned char* q = c ? c + off : nullptr; off += align_up(n, 256); return q; };
  if (kind == L4Q_LORA_QAT) {
    w.wq = take(wq_scratch_bytes(d));
    if (op == L4Q_OP_BWD) w.fac = reinterpret_cast<__half*>(take(factor_scratch_bytes(d)));
  }
  w.v = variant_scratch(p, c ? c + off : nullptr);
  off += w.v.bytes;
  if (kind == L4Q_LORA_QAT) {
    w.zero_B = reinterpret_cast<float*>(take((size_t)p.d_out * p.rank * sizeof(float)));
    if (operand_image_bytes(d, p)) w.op_img = take(operand_image_bytes(d, p));
    if (op == L4Q_OP_BWD) {
      w.dA_unused = reinterpret_cast<float*>(take((size_t)p.rank * p.d_in * sizeof(float)));
      w.dB_unused = reinterpret_cast<float*>(take((size_t)p.d_out * p.rank * sizeof(float)));
      if (wgrad_copy_bytes(d, p)) w.copies = take(wgrad_copy_bytes(d, p));
    }
  }
  w.bytes = off + 256;
  return w;
}

l4q_status lora_check(const l4q_desc* desc, int kind, Params* p) {
  l4q_status st = make_params(desc, p);
  if (st != L4Q_OK) return st;
  if (kind != L4Q_LORA_PLAIN && kind != L4Q_LORA_QAT) return L4Q_ERR_INVALID_ARG;
  if (desc->io_dtype != L4Q_BF16 || p->rank > LORA_PAD) return L4Q_ERR_UNSUPPORTED;
  return L4Q_OK;
}

}  // namespace

extern "C" {

size_t l4q_workspace_bytes(const l4q_desc* desc, int op) {
  Params p;
  if (make_params(desc, &p) != L4Q_OK) return 0;
  switch (op) {
    case L4Q_OP_FWD:
      return wq_scratch_bytes(desc) + operand_image_bytes(desc, p) + 256;
    case L4Q_OP_BWD:   // W_q for the input gradient, and in bf16 mode the fp16 STE factors for the weight gradient
      return wq_scratch_bytes(desc) + (desc->io_dtype == L4Q_BF16 ? factor_scratch_bytes(desc) : 0) +
             operand_image_bytes(desc, p) + wgrad_copy_bytes(desc, p) + 256;
    case L4Q_OP_PACK:   // optional (see l4q_pack_int)
      return operand_image_bytes(desc, p);
    default:
      return 0;
  }
}

l4q_status l4q_linear_fwd(const l4q_desc* desc, const void* X, const void* W0, const float* A, const float* B,
                          const float* s, const float* b, void* Y, void* workspace, size_t workspace_bytes,
                          void* cuda_stream) {
  Params p;
  l4q_status st = make_params(desc, &p);
  if (st != L4Q_OK) return st;
  if (!X || !W0 || !A || !B || !s || !b || !Y) return L4Q_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(W0) || !aligned16(A) || !aligned16(B) || !aligned16(Y)) return L4Q_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < l4q_workspace_bytes(desc, L4Q_OP_FWD) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return L4Q_ERR_WORKSPACE;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  void* wq = workspace;
  if (desc->io_dtype == L4Q_F32) {
    st = launch_dequant<false>(p, W0, A, B, s, b, wq, nullptr, stream);
    if (st != L4Q_OK) return st;
    GemmView g;
    g.A = reinterpret_cast<const float*>(X); g.a_m = p.d_in; g.a_k = 1;
    g.B = reinterpret_cast<const float*>(wq); g.b_k = 1; g.b_n = p.d_in;
    g.M = p.tokens; g.N = p.d_out; g.K = p.d_in;
    dim3 grid(ceil_div(g.N, VT), ceil_div(g.M, VT));
    KernelScope ks(L4Q_KERNEL_VAL_GEMM, stream);
    k_val_gemm<<<grid, V_THREADS, 0, stream>>>(g, reinterpret_cast<float*>(Y));
    return launch_status();
  }
  // the split operands of the merge follow W_q in the workspace
  void* op_img = operand_image_bytes(desc, p) ? static_cast<unsigned char*>(workspace) + wq_scratch_bytes(desc) : nullptr;
  st = launch_dequant<true>(p, W0, A, B, s, b, wq, nullptr, stream, op_img);
  if (st != L4Q_OK) return st;
  KernelScope ks(L4Q_KERNEL_GEMM_FWD, stream);
  return gemm_forward_bf16(p, X, wq, Y, stream);
}

l4q_status l4q_linear_bwd(const l4q_desc* desc, const void* X, const void* dY, const void* W0, const float* A,
                          const float* B, const float* s, const float* b, void* dX, float* dA, float* dB,
                          float* ds, float* db, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  Params p;
  l4q_status st = make_params(desc, &p);
  if (st != L4Q_OK) return st;
  if (!X || !dY || !W0 || !A || !B || !s || !b) return L4Q_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(dY) || !aligned16(W0) || !aligned16(A) || !aligned16(B) || !aligned16(dX))
    return L4Q_ERR_INVALID_ARG;
  const int n_param_out = (dA != nullptr) + (dB != nullptr) + (ds != nullptr) + (db != nullptr);
  if (n_param_out != 0 && n_param_out != 4) return L4Q_ERR_INVALID_ARG;
  const bool f32 = desc->io_dtype == L4Q_F32;
  if (!f32 && n_param_out == 4 && !wgrad_rank_supported(p.rank)) return L4Q_ERR_UNSUPPORTED;
  if (!workspace || workspace_bytes < l4q_workspace_bytes(desc, L4Q_OP_BWD) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return L4Q_ERR_WORKSPACE;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  void* wq = workspace;

  // the reductions below accumulate with fp32 atomics: dA, dB, ds, db start from zero.  The operand split of the
  // recompute step clears them where it runs; otherwise four memsets do.
  const size_t gn = (size_t)p.d_out * p.ngroups;
  const ZeroList grads{{dA, dB, ds, db}, {(size_t)p.rank * p.d_in, (size_t)p.d_out * p.rank, gn, gn}};
  bool zeroed = false;
  // recompute step (App. E.2): W_q for dX and, on the tensor-core path, the STE factors for the weight gradient
  __half* fac = (!f32 && n_param_out == 4)
                    ? reinterpret_cast<__half*>(static_cast<unsigned char*>(workspace) + wq_scratch_bytes(desc))
                    : nullptr;
  unsigned char* ws_tail = static_cast<unsigned char*>(workspace) + wq_scratch_bytes(desc) +
                           (f32 ? 0 : factor_scratch_bytes(desc));
  Bf16Copies copies{};
  bool copied = false;
  if (!f32 && n_param_out == 4) copies = carve_copies(p, ws_tail + operand_image_bytes(desc, p));
  if (dX || fac) {
    st = f32 ? launch_dequant<false>(p, W0, A, B, s, b, wq, nullptr, stream)
             : launch_dequant<true>(p, W0, A, B, s, b,
                                    // W_q is only needed for the input gradient (the plain-ALU kernel always writes it)
                                    (dX || !wtile_tc_supported(p, WT2_FACTORS)) ? wq : nullptr, fac, stream,
                                    operand_image_bytes(desc, p) ? ws_tail : nullptr,
                                    n_param_out == 4 ? &grads : nullptr, &zeroed, fac ? &copies : nullptr, &copied);
    if (st != L4Q_OK) return st;
  }
  if (n_param_out == 4 && !zeroed) {
    if (cudaMemsetAsync(dA, 0, grads.n[0] * sizeof(float), stream) != cudaSuccess ||
        cudaMemsetAsync(dB, 0, grads.n[1] * sizeof(float), stream) != cudaSuccess ||
        cudaMemsetAsync(ds, 0, grads.n[2] * sizeof(float), stream) != cudaSuccess ||
        cudaMemsetAsync(db, 0, grads.n[3] * sizeof(float), stream) != cudaSuccess)
      return cuda_fail();
  }
  if (f32) {
    if (dX) {
      GemmView g;
      g.A = reinterpret_cast<const float*>(dY); g.a_m = p.d_out; g.a_k = 1;
      g.B = reinterpret_cast<const float*>(wq); g.b_k = p.d_in; g.b_n = 1;
      g.M = p.tokens; g.N = p.d_in; g.K = p.d_out;
      dim3 grid(ceil_div(g.N, VT), ceil_div(g.M, VT));
      KernelScope ks(L4Q_KERNEL_VAL_GEMM, stream);
      k_val_gemm<<<grid, V_THREADS, 0, stream>>>(g, reinterpret_cast<float*>(dX));
      if ((st = launch_status()) != L4Q_OK) return st;
    }
    if (n_param_out == 4) {
      dim3 grid(ceil_div(p.d_in, VT), ceil_div(p.d_out, VT));
      KernelScope ks(L4Q_KERNEL_VAL_WGRAD, stream);
      k_val_wgrad<<<grid, V_THREADS, 0, stream>>>(p, reinterpret_cast<const float*>(X),
                                                  reinterpret_cast<const float*>(dY),
                                                  reinterpret_cast<const float*>(W0), A, B, s, b, dA, dB, ds, db);
      if ((st = launch_status()) != L4Q_OK) return st;
    }
    return L4Q_OK;
  }
  if (dX) {
    KernelScope ks(L4Q_KERNEL_GEMM_DGRAD, stream);
    st = gemm_dgrad_bf16(p, dY, wq, dX, stream);
    if (st != L4Q_OK) return st;
  }
  if (n_param_out == 4) {
    if (!copied && (st = launch_copies(p, A, B, copies, stream)) != L4Q_OK) return st;
    KernelScope ks(L4Q_KERNEL_GEMM_WGRAD, stream);
    st = gemm_wgrad_bf16(p, X, dY, fac, copies.A16, copies.Bt16, dA, dB, ds, db, stream);
    if (st != L4Q_OK) return st;
  }
  return L4Q_OK;
}

size_t l4q_lora_workspace_bytes(const l4q_desc* desc, int kind, int op) {
  Params p;
  if (lora_check(desc, kind, &p) != L4Q_OK || (op != L4Q_OP_FWD && op != L4Q_OP_BWD)) return 0;
  return lora_workspace(desc, p, kind, op, nullptr).bytes;
}

l4q_status l4q_lora_linear_fwd(const l4q_desc* desc, int kind, const void* X, const void* W0, const float* A,
                               const float* B, const float* s, const float* b, void* Y, void* workspace,
                               size_t workspace_bytes, void* cuda_stream) {
  Params p;
  l4q_status st = lora_check(desc, kind, &p);
  if (st != L4Q_OK) return st;
  const bool qat = kind == L4Q_LORA_QAT;
  if (!X || !W0 || !A || !B || !Y || (qat && (!s || !b))) return L4Q_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(W0) || !aligned16(A) || !aligned16(B) || !aligned16(Y)) return L4Q_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < l4q_lora_workspace_bytes(desc, kind, L4Q_OP_FWD) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return L4Q_ERR_WORKSPACE;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const LoraWorkspace w = lora_workspace(desc, p, kind, L4Q_OP_FWD, workspace);
  const void* W = W0;
  if (qat) {
    if (cudaMemsetAsync(w.zero_B, 0, (size_t)p.d_out * p.rank * sizeof(float), stream) != cudaSuccess)
      return cuda_fail();
    if ((st = launch_dequant<true>(p, W0, A, w.zero_B, s, b, w.wq, nullptr, stream, w.op_img)) != L4Q_OK) return st;
    W = w.wq;
  }
  {
    KernelScope ks(L4Q_KERNEL_LORA_SIDE, stream);
    if ((st = launch_lora_cast(p, A, B, w.v, stream)) != L4Q_OK) return st;
  }
  {
    KernelScope ks(L4Q_KERNEL_LORA_SIDE, stream);
    if ((st = gemm_lora_down_bf16(p, X, w.v, stream)) != L4Q_OK) return st;
  }
  KernelScope ks(L4Q_KERNEL_GEMM_FWD, stream);
  return gemm_forward_lora_bf16(p, X, W, w.v, Y, stream);
}

l4q_status l4q_lora_linear_bwd(const l4q_desc* desc, int kind, const void* X, const void* dY, const void* W0,
                               const float* A, const float* B, const float* s, const float* b, void* dX, float* dA,
                               float* dB, float* ds, float* db, void* workspace, size_t workspace_bytes,
                               void* cuda_stream) {
  Params p;
  l4q_status st = lora_check(desc, kind, &p);
  if (st != L4Q_OK) return st;
  const bool qat = kind == L4Q_LORA_QAT;
  if (!X || !dY || !W0 || !A || !B || (qat && (!s || !b))) return L4Q_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(dY) || !aligned16(W0) || !aligned16(A) || !aligned16(B) || !aligned16(dX))
    return L4Q_ERR_INVALID_ARG;
  if ((dA != nullptr) != (dB != nullptr) || (ds != nullptr) != (db != nullptr)) return L4Q_ERR_INVALID_ARG;
  if (!qat && ds) return L4Q_ERR_INVALID_ARG;                  // plain LoRA has no quantizer
  if (qat && ds && !wgrad_rank_supported(p.rank)) return L4Q_ERR_UNSUPPORTED;
  if (!workspace || workspace_bytes < l4q_lora_workspace_bytes(desc, kind, L4Q_OP_BWD) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return L4Q_ERR_WORKSPACE;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const LoraWorkspace w = lora_workspace(desc, p, kind, L4Q_OP_BWD, workspace);
  const void* W = W0;
  if (qat && (dX || ds)) {
    if (cudaMemsetAsync(w.zero_B, 0, (size_t)p.d_out * p.rank * sizeof(float), stream) != cudaSuccess)
      return cuda_fail();
    if ((st = launch_dequant<true>(p, W0, A, w.zero_B, s, b, w.wq, ds ? w.fac : nullptr, stream, w.op_img)) != L4Q_OK)
      return st;
    W = w.wq;
  }
  if (dX || dA) {
    {
      KernelScope ks(L4Q_KERNEL_LORA_SIDE, stream);
      if ((st = launch_lora_cast(p, A, B, w.v, stream)) != L4Q_OK) return st;
    }
    KernelScope ks(L4Q_KERNEL_LORA_SIDE, stream);
    if ((st = gemm_lora_up_t_bf16(p, dY, w.v, stream)) != L4Q_OK) return st;         // dYt = dY B
  }
  if (dX) {
    KernelScope ks(L4Q_KERNEL_GEMM_DGRAD, stream);
    if ((st = gemm_dgrad_lora_bf16(p, dY, W, w.v, dX, stream)) != L4Q_OK) return st;
  }
  if (dA) {
    if (cudaMemsetAsync(dA, 0, (size_t)p.rank * p.d_in * sizeof(float), stream) != cudaSuccess ||
        cudaMemsetAsync(dB, 0, (size_t)p.d_out * p.rank * sizeof(float), stream) != cudaSuccess)
      return cuda_fail();
    {
      KernelScope ks(L4Q_KERNEL_LORA_SIDE, stream);                                  // Xt = X A^T, recomputed
      if ((st = gemm_lora_down_bf16(p, X, w.v, stream)) != L4Q_OK) return st;
    }
    {
      KernelScope ks(L4Q_KERNEL_LORA_SIDE, stream);
      if ((st = gemm_lora_da_bf16(p, X, w.v, dA, stream)) != L4Q_OK) return st;
    }
    KernelScope ks(L4Q_KERNEL_LORA_SIDE, stream);
    if ((st = gemm_lora_db_bf16(p, dY, w.v, dB, stream)) != L4Q_OK) return st;
  }
  if (qat && ds) {
    const size_t gsz = (size_t)p.d_out * p.ngroups * sizeof(float);
    if (cudaMemsetAsync(ds, 0, gsz, stream) != cudaSuccess || cudaMemsetAsync(db, 0, gsz, stream) != cudaSuccess)
      return cuda_fail();
    const Bf16Copies cp = carve_copies(p, w.copies);
    if ((st = launch_copies(p, A, w.zero_B, cp, stream)) != L4Q_OK) return st;
    KernelScope ks(L4Q_KERNEL_GEMM_WGRAD, stream);
    if ((st = gemm_wgrad_bf16(p, X, dY, w.fac, cp.A16, cp.Bt16, w.dA_unused, w.dB_unused, ds, db, stream)) != L4Q_OK)
      return st;
  }
  return L4Q_OK;
}

l4q_status l4q_pack_int(const l4q_desc* desc, const void* W0, const float* A, const float* B, const float* s,
                        const float* b, uint32_t* codes, uint16_t* s_fp16, uint16_t* b_fp16, void* workspace,
                        size_t workspace_bytes, void* cuda_stream) {
  Params p;
  l4q_status st = make_params(desc, &p);
  if (st != L4Q_OK) return st;
  if (!W0 || !A || !B || !s || !b || !codes || !s_fp16 || !b_fp16) return L4Q_ERR_INVALID_ARG;
  if (!aligned16(W0) || !aligned16(A) || !aligned16(codes)) return L4Q_ERR_INVALID_ARG;
  if (p.bits != 3 && p.bits != 4) return L4Q_ERR_UNSUPPORTED;
  if (((int64_t)p.d_in * p.bits) % 32 != 0) return L4Q_ERR_UNSUPPORTED;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  __half* s16 = reinterpret_cast<__half*>(s_fp16);
  __half* b16 = reinterpret_cast<__half*>(b_fp16);
  // the workspace is optional: with it the split operands of the merge are built once instead of tile by tile
  const size_t img = operand_image_bytes(desc, p);
  void* op_img = (workspace && img && workspace_bytes >= img && !(reinterpret_cast<uintptr_t>(workspace) & 255u))
                     ? workspace : nullptr;
  return desc->io_dtype == L4Q_BF16 ? launch_pack<true>(p, W0, A, B, s, b, codes, s16, b16, stream, op_img)
                                    : launch_pack<false>(p, W0, A, B, s, b, codes, s16, b16, stream);
}

l4q_status l4q_linear_infer(const l4q_desc* desc, const void* X, const uint32_t* codes, const uint16_t* s_fp16,
                            const uint16_t* b_fp16, void* Y, void* cuda_stream) {
  if (!desc) return L4Q_ERR_INVALID_ARG;
  l4q_desc d2 = *desc;
  d2.rank = 8; d2.alpha = 1.f; d2.grad_scale = 1.f;                     // unused by this op
  Params p;
  l4q_status st = make_params(&d2, &p);
  if (st != L4Q_OK) return st;
  if (!X || !codes || !s_fp16 || !b_fp16 || !Y) return L4Q_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(codes) || !aligned16(Y)) return L4Q_ERR_INVALID_ARG;
  if (desc->io_dtype != L4Q_BF16 || !infer_supported(p)) return L4Q_ERR_UNSUPPORTED;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  KernelScope ks(L4Q_KERNEL_INFER, stream);
  if (gemv_supported(p))                                                 // 1 or 2 tokens: matrix-vector kernel
    return launch_infer_gemv(p, X, codes, reinterpret_cast<const __half*>(s_fp16),
                             reinterpret_cast<const __half*>(b_fp16), Y, stream);
  return launch_infer_bf16(p, X, codes, reinterpret_cast<const __half*>(s_fp16),
                           reinterpret_cast<const __half*>(b_fp16), Y, stream);
}

l4q_status l4q_adamw_step(float* param, const float* grad, float* m, float* v, size_t n, int64_t step, float lr,
                          float beta1, float beta2, float eps, float weight_decay, void* cuda_stream) {
  if (!param || !grad || !m || !v || n == 0 || step < 1) return L4Q_ERR_INVALID_ARG;
  if (!(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps >= 0.f) || !(lr == lr))
    return L4Q_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const double c1 = 1.0 - std::pow((double)beta1, (double)step), c2 = 1.0 - std::pow((double)beta2, (double)step);
  const int blocks = (int)std::min<size_t>((n + 255) / 256, (size_t)sm_count() * 8);
  KernelScope ks(L4Q_KERNEL_ADAMW, stream);
  k_adamw<<<blocks, 256, 0, stream>>>(param, grad, m, v, n, lr, beta1, beta2, eps, weight_decay, (float)(1.0 / c1),
                                      (float)(1.0 / c2));
  return launch_status();
}

l4q_status l4q_adamw_step_multi(const l4q_adamw_tensor* tensors, int count, int64_t step, float lr, float beta1,
                                float beta2, float eps, float weight_decay, void* cuda_stream) {
  if (!tensors || count < 1 || count > ADAMW_MAX_TENSORS || step < 1) return L4Q_ERR_INVALID_ARG;
  if (!(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps >= 0.f) || !(lr == lr))
    return L4Q_ERR_INVALID_ARG;
  AdamwTable t{};
  unsigned long long total = 0;
  for (int k = 0; k < count; ++k) {
    const l4q_adamw_tensor& x = tensors[k];
    if (!x.param || !x.grad || !x.m || !x.v || x.n == 0) return L4Q_ERR_INVALID_ARG;
    t.param[k] = x.param; t.grad[k] = x.grad; t.m[k] = x.m; t.v[k] = x.v;
    total += x.n;
    t.end[k] = total;
  }
  t.count = count;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const double c1 = 1.0 - std::pow((double)beta1, (double)step), c2 = 1.0 - std::pow((double)beta2, (double)step);
  const int blocks = (int)std::min<unsigned long long>((total + 255) / 256, (unsigned long long)sm_count() * 8);
  KernelScope ks(L4Q_KERNEL_ADAMW, stream);
  k_adamw_multi<<<blocks, 256, 0, stream>>>(t, lr, beta1, beta2, eps, weight_decay, (float)(1.0 / c1), (float)(1.0 / c2));
  return launch_status();
}

l4q_status l4q_init_params(const l4q_desc* desc, const void* W, int method, float* s, float* b, void* cuda_stream) {
  l4q_desc d2;
  if (!desc) return L4Q_ERR_INVALID_ARG;
  d2 = *desc;
  d2.tokens = 1; d2.rank = 8; d2.alpha = 1.f; d2.grad_scale = 1.f;      // unused by this op
  Params p;
  l4q_status st = make_params(&d2, &p);
  if (st != L4Q_OK) return st;
  if (!W || !s || !b || !aligned16(W)) return L4Q_ERR_INVALID_ARG;
  if (method < L4Q_INIT_LSQ_PLUS || method > L4Q_INIT_L4Q) return L4Q_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const long long groups = (long long)p.d_out * p.ngroups;
  const int blocks = (int)std::min<long long>((groups + 7) / 8, (long long)sm_count() * 16);
  const bool signed_grid = (desc->flags & L4Q_FLAG_SIGNED_GRID) != 0;
  KernelScope ks(L4Q_KERNEL_INIT, stream);
  if (desc->io_dtype == L4Q_BF16 && init_tma_supported(p)) return launch_init_tma(p, method, signed_grid, W, s, b, stream);
  int lanes_log2 = -1;                                   // group = 8 * 2^k elements with k <= 5: the coalesced kernel
  for (int k = 0; k <= 5; ++k)
    if (p.group == (8 << k)) lanes_log2 = k;
  if (lanes_log2 >= 0) {
    const long long pieces = (long long)p.d_out * p.d_in / 8;
    const int vblocks = (int)std::min<long long>((pieces + 1023) / 1024, 1LL << 20);   // one sweep: blocks balance themselves
    if (desc->io_dtype == L4Q_BF16)
      k_init_params_vec<true><<<vblocks, 256, 0, stream>>>(p, method, signed_grid, lanes_log2, W, s, b);
    else
      k_init_params_vec<false><<<vblocks, 256, 0, stream>>>(p, method, signed_grid, lanes_log2, W, s, b);
    return launch_status();
  }
  if (desc->io_dtype == L4Q_BF16) k_init_params<true><<<blocks, 256, 0, stream>>>(p, method, signed_grid, W, s, b);
  else k_init_params<false><<<blocks, 256, 0, stream>>>(p, method, signed_grid, W, s, b);
  return launch_status();
}

l4q_status l4q_quant_error(const l4q_desc* desc, const void* W0, const float* A, const float* B, const float* s,
                           const float* b, double* errors, void* cuda_stream) {
  Params p;
  l4q_status st = make_params(desc, &p);
  if (st != L4Q_OK) return st;
  if (!W0 || !A || !B || !s || !b || !errors) return L4Q_ERR_INVALID_ARG;
  if (!aligned16(W0) || !aligned16(A) || (reinterpret_cast<uintptr_t>(errors) & 7u)) return L4Q_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(errors, 0, 2 * sizeof(double), stream) != cudaSuccess) return cuda_fail();
  if (desc->io_dtype == L4Q_BF16 && wtile_tc_supported(p, WT2_ERROR)) {   // tensor-core merge, W0 by TMA; no scratch:
    KernelScope ks(L4Q_KERNEL_ERROR, stream);                              // one warp builds the merge operands
    return launch_wtile_tc(WT2_ERROR, p, W0, A, B, s, b, nullptr, nullptr, nullptr, nullptr, stream, nullptr, nullptr,
                           nullptr, nullptr, errors);
  }
  const size_t smem = weight_tile_smem_bytes(p.rank);
  dim3 grid(ceil_div(p.d_in, WT_COLS), ceil_div(p.d_out, WT_ROWS));
  auto launch = [&](auto kern) -> l4q_status {
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return cuda_fail();
    KernelScope ks(L4Q_KERNEL_ERROR, stream);
    kern<<<grid, WT_THREADS, smem, stream>>>(p, W0, A, B, s, b, nullptr, nullptr, nullptr, nullptr, nullptr, errors);
    return launch_status();
  };
  return desc->io_dtype == L4Q_BF16 ? launch(k_weight_tile<true, WT_MODE_ERROR>)
                                    : launch(k_weight_tile<false, WT_MODE_ERROR>);
}

// ---- forward without caller-provided scratch --------------------------------------------------
// Scratch for the dequantized weight of l4q_linear_fwd_static.  Lives in the library image: every
// device that loads the library reserves these bytes until the process exits.
static __device__ __align__(256) unsigned char g_fwd_static_scratch[L4Q_STATIC_SCRATCH_BYTES];

// Never launched; naming the array in device code keeps the symbol in the device image.
__global__ void k_static_scratch_anchor(unsigned char* out) {
  if (out) *out = g_fwd_static_scratch[0];
}

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void* g_static_ptr[kMaxDevices];   // device address of g_fwd_static_scratch, per device; null until set up

// In host code `g_fwd_static_scratch` is only a handle for the runtime, not an address a kernel can
// use.  The device address is looked up once per device, with that device current.
l4q_status static_scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cuda_fail();
  std::lock_guard<std::mutex> lk(g_static_mu);
  if (!g_static_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_fwd_static_scratch) != cudaSuccess || !ptr) return cuda_fail();
    g_static_ptr[dev] = ptr;
  }
  *out = g_static_ptr[dev];
  return L4Q_OK;
}
}  // namespace

l4q_status l4q_linear_fwd_static(const l4q_desc* desc, const void* X, const void* W0, const float* A, const float* B,
                                 const float* s, const float* b, void* Y, void* cuda_stream) {
  Params p;
  l4q_status st = make_params(desc, &p);
  if (st != L4Q_OK) return st;
  if (!X || !W0 || !A || !B || !s || !b || !Y) return L4Q_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(W0) || !aligned16(A) || !aligned16(B) || !aligned16(Y)) return L4Q_ERR_INVALID_ARG;
  if (wq_scratch_bytes(desc) > (size_t)L4Q_STATIC_SCRATCH_BYTES) return L4Q_ERR_WORKSPACE;   // weight too large
  void* wq = nullptr;
  if ((st = static_scratch_for_current_device(&wq)) != L4Q_OK) return st;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  // The whole d_out x d_in region that the GEMM reads is rewritten by the dequantize kernel first,
  // so nothing left in the array by an earlier call is ever read.
  if (desc->io_dtype == L4Q_F32) {
    st = launch_dequant<false>(p, W0, A, B, s, b, wq, nullptr, stream);
    if (st != L4Q_OK) return st;
    GemmView g;
    g.A = reinterpret_cast<const float*>(X); g.a_m = p.d_in; g.a_k = 1;
    g.B = reinterpret_cast<const float*>(wq); g.b_k = 1; g.b_n = p.d_in;
    g.M = p.tokens; g.N = p.d_out; g.K = p.d_in;
    dim3 grid(ceil_div(g.N, VT), ceil_div(g.M, VT));
    KernelScope ks(L4Q_KERNEL_VAL_GEMM, stream);
    k_val_gemm<<<grid, V_THREADS, 0, stream>>>(g, reinterpret_cast<float*>(Y));
    return launch_status();
  }
  st = launch_dequant<true>(p, W0, A, B, s, b, wq, nullptr, stream);
  if (st != L4Q_OK) return st;
  KernelScope ks(L4Q_KERNEL_GEMM_FWD, stream);
  return gemm_forward_bf16(p, X, wq, Y, stream);
}

l4q_status l4q_selftest_timeout(void* cuda_stream) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  k_selftest_timeout<<<1, 32, 0, stream>>>();
  return launch_status();
}

l4q_status l4q_selftest_tile_copy(const void* src, void* dst, int64_t rows, int64_t cols, void* cuda_stream) {
  if (!src || rows <= 0 || cols <= 0 || rows > (1 << 30) || cols > (1 << 30) || cols % 8 != 0) return L4Q_ERR_INVALID_ARG;
  if (!aligned16(src) || !aligned16(dst)) return L4Q_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  KernelScope ks(L4Q_KERNEL_TILE_COPY, stream);
  return launch_tile_copy(src, dst, (int)rows, (int)cols, stream);
}

l4q_status l4q_check(void* cuda_stream) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (cudaStreamSynchronize(stream) != cudaSuccess) return cuda_fail();
  unsigned int word = 0;
  if (cudaMemcpyFromSymbol(&word, g_l4q_status, sizeof(word)) != cudaSuccess) return cuda_fail();
  if (word != 0) {
    const unsigned int zero = 0;
    if (cudaMemcpyToSymbol(g_l4q_status, &zero, sizeof(zero)) != cudaSuccess) return cuda_fail();
    return (l4q_status)word;
  }
  return L4Q_OK;
}

uint64_t l4q_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

l4q_status l4q_profile_enable(int enable) {
  std::lock_guard<std::mutex> lk(g_prof_mu);
  if (enable && g_prof_pool.empty()) {
    g_prof_pool.resize(kProfPool);
    for (auto& sl : g_prof_pool) {
      if (cudaEventCreate(&sl.begin) != cudaSuccess || cudaEventCreate(&sl.end) != cudaSuccess) {
        g_prof_pool.clear();
        return cuda_fail();
      }
    }
  }
  if (enable && !g_prof_on) {
    g_prof_used = 0;
    for (int k = 0; k < L4Q_KERNEL_COUNT; ++k) { g_prof_ms[k] = 0.0; g_prof_n[k] = 0; }
  }
  if (!enable && g_prof_on) prof_drain_locked();
  g_prof_on = enable != 0;
  return L4Q_OK;
}

l4q_status l4q_profile_read(int kernel, uint64_t* launches, double* total_ms) {
  if (kernel < 0 || kernel >= L4Q_KERNEL_COUNT || !launches || !total_ms) return L4Q_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(g_prof_mu);
  prof_drain_locked();
  *launches = g_prof_n[kernel];
  *total_ms = g_prof_ms[kernel];
  return L4Q_OK;
}

const char* l4q_kernel_name(int kernel) {
  switch (kernel) {
    case L4Q_KERNEL_DEQUANT: return "weight tile: merge + fake-quantize";
    case L4Q_KERNEL_PACK: return "weight tile: merge + quantize + pack";
    case L4Q_KERNEL_GEMM_FWD: return "k_gemm_bf16<fwd>";
    case L4Q_KERNEL_GEMM_DGRAD: return "k_gemm_bf16<dgrad>";
    case L4Q_KERNEL_GEMM_WGRAD: return "k_gemm_bf16<wgrad>";
    case L4Q_KERNEL_VAL_GEMM: return "k_val_gemm";
    case L4Q_KERNEL_VAL_WGRAD: return "k_val_wgrad";
    case L4Q_KERNEL_INIT: return "k_init_params";
    case L4Q_KERNEL_ERROR: return "k_weight_tile<error sums>";
    case L4Q_KERNEL_INFER: return "k_infer_bf16";
    case L4Q_KERNEL_ADAMW: return "k_adamw";
    case L4Q_KERNEL_LORA_SIDE: return "k_gemm_bf16<rank side> / k_lora_cast";
    case L4Q_KERNEL_TILE_COPY: return "k_tile_copy";
    default: return "unknown kernel";
  }
}

const char* l4q_status_string(l4q_status status) {
  switch (status) {
    case L4Q_OK: return "ok";
    case L4Q_ERR_INVALID_ARG: return "invalid argument";
    case L4Q_ERR_UNSUPPORTED: return "unsupported shape, bit-width or rank";
    case L4Q_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case L4Q_ERR_CUDA: return "CUDA call failed";
    case L4Q_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

}  // extern "C"
