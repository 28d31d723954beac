/*
 * l4q.h -- C ABI of the B200 (sm_100a) L4Q linear-layer library.
 *
 * The layer (arXiv 2402.04902, Sec. 3.2) merges a frozen weight with a LoRA
 * update, fake-quantizes the merge group-wise with a learnable scale and
 * offset, and multiplies:
 *
 *     gamma  = alpha / rank
 *     W_comb = W0 + gamma * B A                                   (Eq. 7)
 *     w      = (W_comb - b) / s           per group of `group_size`
 *                                         consecutive elements of a row
 *     w~     = round(clamp(w, Q_N, Q_P))                          (Eq. 8)
 *     W_q    = w~ * s + b                                         (Eq. 9)
 *     Y      = X W_q^T                                            (Eq. 10)
 *
 * Layout: every tensor is dense row-major.  tokens = flattened batch x seq.
 *     X [tokens, d_in]   Y, dY [tokens, d_out]   dX [tokens, d_in]
 *     W0 [d_out, d_in]   A [rank, d_in]   B [d_out, rank]
 *     s, b, ds, db [d_out, d_in / group_size]
 * X, Y, dY, dX and W0 have the dtype `io_dtype` (bf16 or fp32); A, B, s, b
 * and every parameter gradient are fp32.
 *
 * Integer grid: by default the codes are unsigned, [Q_N, Q_P] = [0, 2^bits-1];
 * L4Q_FLAG_SIGNED_GRID selects the grid printed in Eq. 3,
 * [-2^(bits-1), 2^(bits-1)-1].  round() is round-half-to-even.
 *
 * Conventions shared by every entry point:
 *   - all tensor pointers are DEVICE pointers owned by the caller, 16-byte
 *     aligned; the library allocates no memory and keeps nothing between
 *     calls (the forward saves nothing for the backward: the backward
 *     recomputes the quantized weight, App. E.2);
 *   - `workspace` is caller-owned device scratch of at least
 *     l4q_workspace_bytes() bytes, 256-byte aligned; its contents are
 *     undefined before and after a call;
 *   - calls are asynchronous on `cuda_stream` (a cudaStream_t, NULL = default
 *     stream); outputs are overwritten, never accumulated into;
 *   - errors are return codes only: no exception, no abort, no device trap.
 *     A device-side wait that runs out of patience records L4Q_ERR_TIMEOUT in
 *     a device status word which l4q_check() reads.
 */
#ifndef L4Q_H_
#define L4Q_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  L4Q_OK = 0,
  L4Q_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, misaligned pointer      */
  L4Q_ERR_UNSUPPORTED = 2,   /* shape / bit-width / rank outside what the kernels cover */
  L4Q_ERR_WORKSPACE = 3,     /* workspace missing or smaller than l4q_workspace_bytes()  */
  L4Q_ERR_CUDA = 4,          /* a CUDA runtime or driver call failed                     */
  L4Q_ERR_TIMEOUT = 5        /* a bounded device-side wait expired (results invalid)     */
} l4q_status;

enum { L4Q_BF16 = 0, L4Q_F32 = 1 };                 /* io_dtype */
enum { L4Q_OP_FWD = 0, L4Q_OP_BWD = 1, L4Q_OP_PACK = 2 };
#define L4Q_MAX_RANK 128   /* largest LoRA rank any entry point takes (else L4Q_ERR_UNSUPPORTED) */
enum {
  L4Q_FLAG_SIGNED_GRID = 1u   /* codes in [-2^(bits-1), 2^(bits-1)-1] as in Eq. 3 */
};

/* Problem statement of one layer (Sec. 2.1, 2.2, 3.2).  Plain data, passed by pointer (host memory). */
typedef struct l4q_desc {
  int64_t  tokens;      /* rows of X / Y                                                   */
  int64_t  d_in;        /* i: columns of W0; multiple of group_size                        */
  int64_t  d_out;       /* o: rows of W0                                                   */
  int32_t  rank;        /* r of the LoRA factors, 1..L4Q_MAX_RANK                          */
  float    alpha;       /* LoRA constant; the merge uses gamma = alpha / rank              */
  int32_t  bits;        /* n: 2..8 for fwd/bwd, 3 or 4 for l4q_pack_int                    */
  int32_t  group_size;  /* g: quantization group along d_in; multiple of 8                 */
  int32_t  io_dtype;    /* L4Q_BF16 or L4Q_F32                                             */
  uint32_t flags;       /* L4Q_FLAG_*                                                      */
  float    grad_scale;  /* multiplies ds and db; 1.0f reproduces the paper                 */
} l4q_desc;

/* Bytes of device scratch the given op (L4Q_OP_*) needs for this problem; 0 if desc is invalid. */
size_t l4q_workspace_bytes(const l4q_desc* desc, int op);

/*
 * Forward, Eq. 7-10: Y = X Q(W0 + gamma B A)^T.
 * In: X, W0 (io_dtype), A, B, s, b (fp32).  Out: Y (io_dtype), overwritten.
 * bf16 mode: W_q is rounded to bf16 and the product accumulates in fp32 on the
 * tensor cores; fp32 mode is a plain-ALU validation path.
 */
l4q_status l4q_linear_fwd(const l4q_desc* desc, const void* X, const void* W0,
                          const float* A, const float* B, const float* s, const float* b,
                          void* Y, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Backward.  Recomputes W_q from (W0, A, B, s, b); takes nothing from the forward.
 *   dX = dY W_q                                   (linear backward implied by Eq. 10)
 *   G  = dY^T X                                   (Eq. 11; never written to memory as a whole)
 *   m  = [Q_N <= w <= Q_P]                        (App. A.1, inclusive, on the unrounded w; each
 *                                                  bound is widened by 2^-10 of a quantization step,
 *                                                  so an element that a min/max initialisation puts
 *                                                  exactly on a bound counts as in range, cf. Table 4)
 *   ds = grad_scale * sum_group G * {Q_N if w<Q_N | w~ - w if m | Q_P if w>Q_P}   (Eq. 5, App. A.1)
 *   db = grad_scale * sum_group G * (1 - m)                                       (Eq. 6, App. A.1)
 *   dA = gamma * B^T (G*m)                        (Eq. 13, App. A.2)
 *   dB = gamma * (G*m) A^T                        (Eq. 14, App. A.2)
 * Any of dX, dA, dB, ds, db may be NULL to skip it (dA, dB, ds, db are produced
 * together: pass all four or none).  Outputs are overwritten.
 * dA, dB, ds, db are sums over tiles of G that the bf16 path accumulates with fp32 atomic adds: their last bits
 * depend on the order in which the tiles finish and differ from run to run (relative differences of ~1e-6, far
 * inside the 3e-2 comparison tolerance).  There is no deterministic mode: it would need the per-tile partial sums
 * in the workspace (d_out/128 copies of dA, d_in/256 copies of dB) and a second reduction pass over them, which is
 * more memory traffic than the reduction itself.  dX and Y do not depend on any order.
 */
l4q_status l4q_linear_bwd(const l4q_desc* desc, const void* X, const void* dY, const void* W0,
                          const float* A, const float* B, const float* s, const float* b,
                          void* dX, float* dA, float* dB, float* ds, float* db,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Export of the fully quantized layer (Sec. 3.2: inference keeps only w~, s, b).
 * The paper fixes no storage format; this library's is:
 *   u = w~ - Q_N in [0, 2^bits - 1]; code j of a row occupies bits
 *   [j*bits, (j+1)*bits) of the row's bitstream, least significant bit first,
 *   stored as little-endian 32-bit words: codes [d_out, d_in*bits/32] (uint32);
 *   s_fp16 = fp16(s), b_fp16 = fp16(b + s*Q_N) as IEEE binary16 bit patterns
 *   [d_out, d_in/group_size], so that W_q ~= u * s_fp16 + b_fp16.
 * Codes are taken with the fp32 s and b (they equal the forward's codes).
 * bits must be 3 or 4 and d_in*bits a multiple of 32.  The workspace is optional: NULL works; given
 * l4q_workspace_bytes(desc, L4Q_OP_PACK) bytes of 256-byte aligned device scratch the bf16 path is faster
 * (the split LoRA operands of the merge are then built once per call instead of once per tile).
 */
l4q_status l4q_pack_int(const l4q_desc* desc, const void* W0, const float* A, const float* B,
                        const float* s, const float* b,
                        uint32_t* codes, uint16_t* s_fp16, uint16_t* b_fp16,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The two layers L4Q is set against, on the same kernels, for measuring what the merged quantization
 * costs per step (Sec. 3.1; the training-time remark of App. E).  `kind`:
 *   L4Q_LORA_PLAIN  Y = X W0^T + gamma (X A^T) B^T                                          (Eq. 1)
 *                   dA = gamma (dY B)^T X,   dB = gamma dY^T (X A^T)                        (Eq. 2)
 *                   dX = dY W0 + gamma (dY B) A
 *   L4Q_LORA_QAT    QAT-LoRA: the same with W0 replaced by Q(W0) = round(clamp((W0-b)/s)) s + b (Eq. 3),
 *                   and ds, db = the LSQ gradients of that quantizer (Eq. 5-6, App. A.1) from the full
 *                   weight gradient dY^T X; the LoRA factors and the quantizer do not see each other.
 * Same layouts, dtypes and conventions as l4q_linear_fwd / l4q_linear_bwd; io_dtype must be L4Q_BF16
 * and rank <= 64 (else L4Q_ERR_UNSUPPORTED).  s, b are read by L4Q_LORA_QAT only (NULL otherwise).
 * X A^T and dY B are rounded to bf16, as are A and B where a tensor-core product reads them; every
 * product accumulates in fp32.  The backward takes nothing from the forward (X A^T is recomputed).
 * Backward outputs: dX may be NULL; dA and dB come together or not at all; ds and db likewise, and
 * only for L4Q_LORA_QAT (rank 8, 16, 32 or 64) -- passing them with L4Q_LORA_PLAIN is
 * L4Q_ERR_INVALID_ARG.  Outputs are overwritten.  Workspace: l4q_lora_workspace_bytes(desc, kind, op),
 * op = L4Q_OP_FWD or L4Q_OP_BWD (0 if the problem is invalid or unsupported).
 */
enum { L4Q_LORA_PLAIN = 1, L4Q_LORA_QAT = 2 };

size_t l4q_lora_workspace_bytes(const l4q_desc* desc, int kind, int op);

l4q_status l4q_lora_linear_fwd(const l4q_desc* desc, int kind, const void* X, const void* W0,
                               const float* A, const float* B, const float* s, const float* b,
                               void* Y, void* workspace, size_t workspace_bytes, void* cuda_stream);

l4q_status l4q_lora_linear_bwd(const l4q_desc* desc, int kind, const void* X, const void* dY, const void* W0,
                               const float* A, const float* B, const float* s, const float* b,
                               void* dX, float* dA, float* dB, float* ds, float* db,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Inference with the fully quantized layer (Sec. 3.2, App. F): Y = X W_q^T, where the weight is rebuilt
 * on the fly from the export of l4q_pack_int,
 *     W_q[o, j] = u[o, j] * s_fp16[o, j / group_size] + b_fp16[o, j / group_size]     (Eq. 9, unsigned code u)
 * and never exists in memory as a whole (bits / 8 bytes per weight are read).
 * In: X [tokens, d_in] bf16; codes [d_out, d_in * bits / 32] uint32, s_fp16, b_fp16 [d_out, d_in / group_size]
 * exactly as written by l4q_pack_int.  Out: Y [tokens, d_out] bf16, overwritten.  W_q is formed in fp32 (within
 * 2^-12 of a quantization step of u s + b) and rounded once to bf16 for the tensor cores; accumulation is fp32.
 * Meant for the few-token regime of App. F (a step of batch 1..64); larger token counts work (in tiles of 128
 * tokens, each of which reads the weight again).  io_dtype must be L4Q_BF16, bits 3 or 4, group_size a multiple
 * of 32 and d_in * bits / 8 a multiple of 16 (else L4Q_ERR_UNSUPPORTED); rank, alpha and flags are ignored.
 * Needs no workspace.
 */
l4q_status l4q_linear_infer(const l4q_desc* desc, const void* X, const uint32_t* codes, const uint16_t* s_fp16,
                            const uint16_t* b_fp16, void* Y, void* cuda_stream);

/*
 * Initialisation of the quantization parameters from a weight (Sec. 3.3, Eq. 15; App. B).
 * In: W [d_out, d_in] (io_dtype; normally W0).  Out: s, b [d_out, d_in / group_size] (fp32), overwritten.
 * `method` (with Q_N = -2^(bits-1), Q_P = 2^(bits-1) - 1 of Eq. 3, per group):
 *   L4Q_INIT_LSQ_PLUS  s = max(|mu - 3 sigma|, |mu + 3 sigma|) / 2^(bits-1),  b = 0
 *                      (mu, sigma: mean and population standard deviation of the group)
 *   L4Q_INIT_SYMM      s = max|W| / 2^(bits-1),                               b = 0
 *   L4Q_INIT_ASYMM     s = (max W - min W) / (Q_P - Q_N),                     b = min W - s Q_N
 *   L4Q_INIT_L4Q       s = max(|min W / Q_N|, |max W / Q_P|),                 b = 0          (Eq. 15)
 * These are the parameters of the signed grid; without L4Q_FLAG_SIGNED_GRID the same quantizer is
 * written for the grid [0, 2^bits - 1], i.e. b + s Q_N is returned as b (ASYMM: b = min W).
 * s is floored at 1e-8 (a constant group would give s = 0; Eq. 3 needs s > 0).
 * desc->tokens, rank and alpha are ignored.  Needs no workspace.
 */
enum { L4Q_INIT_LSQ_PLUS = 0, L4Q_INIT_SYMM = 1, L4Q_INIT_ASYMM = 2, L4Q_INIT_L4Q = 3 };
l4q_status l4q_init_params(const l4q_desc* desc, const void* W, int method, float* s, float* b, void* cuda_stream);

/*
 * Error sums of Table 4 for the current parameters:
 *   errors[0] = E_quant = sum over all weights of |W_comb - W_q|              (Eq. 7-9)
 *   errors[1] = E_clip  = the part of that sum from weights outside the quantization range, i.e.
 *                         where the STE gate of App. A.1 is closed (same 2^-10 guard band as the backward)
 * (the paper gives the two names and their values, not a formula: this is the reading taken).
 * In: W0 (io_dtype), A, B, s, b (fp32).  Out: errors, two doubles in DEVICE memory, overwritten;
 * accumulated with fp64 atomics from fp32 partial sums, so the last digits depend on the order.
 * Needs no workspace.
 */
l4q_status l4q_quant_error(const l4q_desc* desc, const void* W0, const float* A, const float* B,
                           const float* s, const float* b, double* errors, void* cuda_stream);

/*
 * One AdamW step (App. D: "AdamW ... with a weight decay of 0.01") for one trainable tensor of the layer
 * (A, B, s or b), fused into a single pass over param, grad, m and v (all fp32, n elements, device memory):
 *     p <- p - lr * weight_decay * p
 *     m <- beta1 m + (1 - beta1) g          v <- beta2 v + (1 - beta2) g^2
 *     p <- p - lr * (m / (1 - beta1^step)) / (sqrt(v / (1 - beta2^step)) + eps)
 * `step` counts from 1.  param, m and v are updated in place; grad is read only.
 */
l4q_status l4q_adamw_step(float* param, const float* grad, float* m, float* v, size_t n, int64_t step, float lr,
                          float beta1, float beta2, float eps, float weight_decay, void* cuda_stream);

/*
 * The same AdamW step (App. D) for up to 8 tensors in ONE launch: the trainable tensors of a layer (A, B, s, b)
 * are small, and a launch per tensor is bound by the launch.  `tensors`: HOST array of `count` entries, each with
 * DEVICE pointers to param, grad, m, v (fp32, n elements, n > 0); the entries are read during the call and need
 * not outlive it.  All tensors take the same hyper-parameters and step.  Tensors must not overlap.
 * L4Q_ERR_INVALID_ARG on count outside 1..8, a null pointer, n = 0, step < 1 or betas outside [0, 1).
 */
typedef struct {
  float* param;
  const float* grad;
  float* m;
  float* v;
  size_t n;
} l4q_adamw_tensor;
l4q_status l4q_adamw_step_multi(const l4q_adamw_tensor* tensors, int count, int64_t step, float lr, float beta1,
                                float beta2, float eps, float weight_decay, void* cuda_stream);

/*
 * Forward pass for callers that cannot hand the library any scratch memory.
 * (The paper has no counterpart; this entry point exists for integration only.)
 *
 * Same inputs, output and arithmetic as l4q_linear_fwd, but without the
 * workspace arguments: the dequantized weight goes into a fixed array of
 * L4Q_STATIC_SCRATCH_BYTES that is part of the library's device image.  It is
 * meant for code that runs where device allocation is off limits: a plug-in or
 * custom op inside a runtime whose own allocator has already claimed the
 * device's free memory, a latency-critical loop that must not hit the implicit
 * device-wide synchronisation of cudaMalloc/cudaFree, or a process that is
 * held to a fixed memory budget decided at start-up.  The call performs no
 * cudaMalloc, cudaFree or other allocating call.
 *
 *   - Limit: d_out * d_in * sizeof(io_dtype), rounded up to 256 bytes, must not
 *     exceed L4Q_STATIC_SCRATCH_BYTES (32 MiB: a 4096 x 4096 bf16 weight).
 *     Larger problems return L4Q_ERR_WORKSPACE and launch nothing; use
 *     l4q_linear_fwd with a caller-owned workspace for those.
 *   - Cost: every GPU on which this library is loaded keeps the 32 MiB reserved
 *     until the process exits, whether or not this function is ever called.
 *   - The first call on each device looks up the array's device address (with
 *     that device current) and remembers it; make that first call outside any
 *     stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the last
 *     call left in it.  Nothing in it needs to start at zero (each call
 *     rewrites the whole region it later reads), but two calls whose kernels
 *     can overlap on the GPU (different streams, or different host threads
 *     without ordering) race on it: order them on one stream or with events.
 */
#define L4Q_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
l4q_status l4q_linear_fwd_static(const l4q_desc* desc, const void* X, const void* W0,
                                 const float* A, const float* B, const float* s, const float* b,
                                 void* Y, void* cuda_stream);

/* Exercises the error path of the kernels' bounded waits without touching any data: launches one block that
 * waits on a barrier nothing arrives on, with a limit of about a millisecond.  The wait gives up and the kernel
 * ends normally; the next l4q_check() on the stream returns L4Q_ERR_TIMEOUT (and clears it), after which the
 * library works as before.  No counterpart in the paper.  Returns L4Q_OK if the launch succeeded. */
l4q_status l4q_selftest_timeout(void* cuda_stream);

/* Measurement helper, no counterpart in the paper: moves a dense row-major bf16 matrix `src` [rows, cols]
 * (device pointer, 16-byte aligned, cols a multiple of 8) through shared memory in 128 x 128 tiles with the same
 * TMA loads -- and, if `dst` (same shape, may not overlap src) is not NULL, the same TMA stores -- as the
 * merge + fake-quantize kernel, and does nothing else.  Its device time (l4q_profile_read, L4Q_KERNEL_TILE_COPY)
 * is the floor the memory system sets for a kernel that reads one weight (dst NULL: the export) or reads and
 * rewrites it (the dequantize step) in one launch of that size; bench.py reports the weight-tile kernels against
 * it.  Asynchronous on `cuda_stream`; L4Q_ERR_INVALID_ARG on a bad shape or pointer. */
l4q_status l4q_selftest_tile_copy(const void* src, void* dst, int64_t rows, int64_t cols, void* cuda_stream);

/* Synchronises `cuda_stream`, then returns and clears the device status word
 * (L4Q_OK, or L4Q_ERR_TIMEOUT if a kernel gave up on a bounded wait), or
 * L4Q_ERR_CUDA if the stream reported an error. */
l4q_status l4q_check(void* cuda_stream);

/* Number of kernels launched by this library in this process since load (for launch accounting). */
uint64_t l4q_launch_count(void);

/*
 * Optional per-kernel timing.  While enabled, every kernel this library launches
 * is bracketed by a pair of CUDA events on its stream (a fixed pool of 8192
 * pairs, created on the first enable; launches beyond the pool between two reads
 * are not timed).  l4q_profile_read() waits for the recorded events, adds them
 * to the running totals and returns, for one kernel (L4Q_KERNEL_*), the number
 * of timed launches and their total device time in milliseconds since enabling.
 */
enum {
  L4Q_KERNEL_DEQUANT = 0,     /* merge + fake-quantize -> W_q scratch (Eq. 7-9)             */
  L4Q_KERNEL_PACK = 1,        /* merge + quantize + bit-pack (export)                       */
  L4Q_KERNEL_GEMM_FWD = 2,    /* Y = X W_q^T (Eq. 10)                                       */
  L4Q_KERNEL_GEMM_DGRAD = 3,  /* dX = dY W_q                                                */
  L4Q_KERNEL_GEMM_WGRAD = 4,  /* dY^T X tiles reduced into ds, db, dA, dB (Eq. 11, 5-6, 13-14) */
  L4Q_KERNEL_VAL_GEMM = 5,    /* fp32 validation GEMM                                       */
  L4Q_KERNEL_VAL_WGRAD = 6,   /* fp32 validation weight-gradient reduction                  */
  L4Q_KERNEL_INIT = 7,        /* per-group initialisation of s, b (App. B)                  */
  L4Q_KERNEL_ERROR = 8,       /* E_quant, E_clip sums (Table 4)                             */
  L4Q_KERNEL_INFER = 9,       /* Y = X W_q^T from the packed export (App. F)                */
  L4Q_KERNEL_ADAMW = 10,      /* AdamW update of one parameter tensor (App. D)              */
  L4Q_KERNEL_LORA_SIDE = 11,  /* rank-side products of the LoRA / QAT-LoRA layers (Eq. 1-2) */
  L4Q_KERNEL_TILE_COPY = 12,  /* l4q_selftest_tile_copy (measurement helper)                */
  L4Q_KERNEL_COUNT = 13
};
l4q_status l4q_profile_enable(int enable);
l4q_status l4q_profile_read(int kernel, uint64_t* launches, double* total_ms);
const char* l4q_kernel_name(int kernel);

/* Static, NUL-terminated description of a status code. */
const char* l4q_status_string(l4q_status status);

#ifdef __cplusplus
}
#endif
#endif /* L4Q_H_ */
