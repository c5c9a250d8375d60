/*
 * equiforge.h -- C ABI of the B200 (sm_100a) fused tensor-program library.
 *
 * One entry point per fused program that the paper's equality-saturation
 * superoptimizer rewrites and extracts (Section 7.1 "Workloads": normalisation,
 * MLPs, low-rank adaptation, multi-head attention in decode and prefill).  The
 * library executes those programs; the e-graph search is not part of it.
 *
 * Conventions common to every entry point
 *   - All tensor pointers are DEVICE pointers to bfloat16 data (1-8-7 format),
 *     row-major, contiguous, last dimension fastest, 16-byte aligned.
 *     Arithmetic is bf16 x bf16 -> fp32 accumulate (Figure 4: "acc=f32"); outputs are
 *     rounded to bf16 with round-to-nearest-even.
 *   - `stream` is a cudaStream_t passed as void* (NULL = legacy default stream).
 *     Calls are asynchronous: they enqueue 1..3 kernels and return without synchronising.
 *   - `ws` is a caller-owned DEVICE scratch buffer of at least
 *     ef_<program>_workspace_bytes(...) bytes, 256-byte aligned.  It must be initialised
 *     ONCE with ef_workspace_init() (or zero-filled) before its first use; afterwards the
 *     library keeps its bookkeeping words consistent across calls.  One workspace serves one
 *     call at a time: two calls that may overlap on the GPU need two workspaces.  Apart
 *     from the first 256 bytes (status + bookkeeping) its contents are undefined after a call.
 *   - Ownership: the caller owns every buffer and the stream.  The library allocates no
 *     device memory, frees nothing, and keeps only host-side caches (driver entry point,
 *     kernel attributes, SM count).  Inputs are read-only; the output is fully overwritten.
 *     An output that aliases an input is undefined behaviour.
 *   - Errors: return codes only (no exceptions, no abort, no device trap).  Argument errors
 *     are detected on the host before anything is enqueued.  Every device-side wait is
 *     bounded; a wait that gives up records EF_ERR_DEVICE_TIMEOUT in the workspace status
 *     word, the kernel drains and exits normally, and ef_check_status() reports it.
 *   - There is no CPU fallback: a shape outside the supported set returns
 *     EF_ERR_UNSUPPORTED, a device that is not compute capability 10.x returns EF_ERR_ARCH.
 */
#ifndef EQUIFORGE_H_
#define EQUIFORGE_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    EF_OK = 0,
    EF_ERR_NULL = 1,           /* a required pointer is NULL                                   */
    EF_ERR_SHAPE = 2,          /* non-positive or inconsistent dimensions                      */
    EF_ERR_UNSUPPORTED = 3,    /* valid problem, but no kernel covers it (see each entry)      */
    EF_ERR_ALIGN = 4,          /* pointer not 16-byte aligned (workspace: 256-byte)            */
    EF_ERR_WORKSPACE = 5,      /* ws == NULL or ws_bytes below the query                       */
    EF_ERR_ARCH = 6,           /* current device is not compute capability 10.x                */
    EF_ERR_CUDA = 7,           /* a CUDA runtime/driver call failed; see ef_last_cuda_error()  */
    EF_ERR_DEVICE_TIMEOUT = 8  /* a bounded device-side wait gave up (ef_check_status only)    */
} ef_status;

/* ---- Program 1: fused RMSNorm + matmul ---------------------------------------------------
 * Y = (X * rsqrt(mean(X^2, -1) + eps) * gamma) @ W.
 * Definition: RMSNorm expanded into reduce + pointwise ops feeding a MatMul (Section 7.1,
 * "Implementation"); the per-row factor is invariant along K and is applied after the
 * contraction (Table 1, factor motion; Section 7.2, RMSNorm-MLP discussion), gamma stays on
 * the X side; the sum of squares and the K loop form one fused reduction (Table 1, product
 * fusion); W is partitioned along N and K (Table 1, MatMul refinement "NK").
 *   X [M,K], gamma [K], W [K,N] -> Y [M,N].
 * Supported: 1 <= M <= 16, K % 64 == 0, K <= 4096, N % 8 == 0. */
ef_status ef_rmsnorm_matmul(const void* X, const void* gamma, const void* W, void* Y,
                            int M, int K, int N, float eps,
                            void* ws, size_t ws_bytes, void* stream);
size_t ef_rmsnorm_matmul_workspace_bytes(int M, int K, int N);

/* ---- Program 2: fused gated MLP (SwiGLU) -------------------------------------------------
 * Y = SiLU(X @ Wgate) * (X @ Wup), SiLU(z) = z / (1 + exp(-z)).
 * Definition: the GatedMLP workload of Section 7.1 / Table 2; both projections and the
 * elementwise product run in one kernel (Section 7.2).  K-partitioned partial products are
 * summed (Reduce over the parallel K axis, Table 1 "NK") BEFORE the nonlinear gate.
 *   X [M,K], Wgate [K,N], Wup [K,N] -> Y [M,N].
 * Supported: 1 <= M <= 16, K % 64 == 0, N % 8 == 0. */
ef_status ef_gated_mlp(const void* X, const void* Wgate, const void* Wup, void* Y,
                       int M, int K, int N,
                       void* ws, size_t ws_bytes, void* stream);
size_t ef_gated_mlp_workspace_bytes(int M, int K, int N);

/* ---- Program 2b: RMSNorm fused into the gated MLP (RMSNorm-MLP) ------------------------------
 * Y = SiLU(Xn @ Wgate) * (Xn @ Wup) with Xn = X * rsqrt(mean(X^2,-1) + eps) * gamma.
 * Definition: the RMSNorm-MLP workload (Section 7.2): the per-row normalisation factor moves
 * after each projection, (s (.) X) W == s (.) (X W), and both projections plus the elementwise
 * product run in ONE kernel with no intermediate in global memory.
 *   X [M,K], gamma [K], Wgate [K,N], Wup [K,N] -> Y [M,N].
 * Supported: 1 <= M <= 16, K % 64 == 0, K <= 4096, N % 8 == 0.  Up to 8 rows run as ONE kernel; 9..16
 * rows run as two launches of at most 8 rows each on the same workspace (the operand of the tensor
 * core carries the rounding remainder of x*gamma in spare rows, which exist for at most 8 rows). */
ef_status ef_rmsnorm_gated_mlp(const void* X, const void* gamma, const void* Wgate, const void* Wup, void* Y,
                               int M, int K, int N, float eps,
                               void* ws, size_t ws_bytes, void* stream);
size_t ef_rmsnorm_gated_mlp_workspace_bytes(int M, int K, int N);

/* ---- LayerNorm fused into a projection --------------------------------------------------------
 * Y = LayerNorm(X) @ W,  LayerNorm(x)_k = (x_k - mean) * rsqrt(var + eps) * gamma_k + beta_k with
 * mean and (biased) variance over the row (the paper names the LayerNorm+GEMM workload without
 * defining it, Sections 7.1 and 7.2: this is the standard operator).  The mean subtraction does not
 * commute with the contraction as a row scale, so the operand staged in shared memory is
 * (x - mean) * gamma; the inverse standard deviation is invariant along K and scales the finished
 * projection (Table 1, factor motion); beta @ W is produced by the same MMA from a spare operand
 * row.  One kernel.
 *   X [M,K], gamma [K], beta [K], W [K,N] -> Y [M,N].
 * Supported: M <= 15, K % 64 == 0, K <= 4096, N % 8 == 0. */
ef_status ef_layernorm_matmul(const void* X, const void* gamma, const void* beta, const void* W, void* Y,
                              int M, int K, int N, float eps,
                              void* ws, size_t ws_bytes, void* stream);
size_t ef_layernorm_matmul_workspace_bytes(int M, int K, int N);

/* ---- Program 3: grouped-query decode attention -------------------------------------------
 * One query token per sequence attends all L cached keys: for query head h and kv head
 * g = h / (Hq/Hkv):  O[b,h] = softmax_j(scale * Q[b,h] . K[b,g,j]) @ V[b,g].
 * Definition: vanilla attention M0 of Figure 4, executed as the tiled rolling form M2
 * (state <max,sum,value>, repair h(c,s,s') = c*exp(s-s'), Section 4.2); the key axis is also
 * split across thread blocks and the partial states are stored and merged (Table 1,
 * intermediate storage; Section 4.4).
 *   Q [B,Hq,D], K [B,Hkv,L,D], V [B,Hkv,L,D] -> O [B,Hq,D].
 * Supported: D == 128, Hq % Hkv == 0, Hq/Hkv <= 8, L >= 1. */
ef_status ef_gqa_decode(const void* Q, const void* K, const void* V, void* O,
                        int B, int Hq, int Hkv, int L, int D, float scale,
                        void* ws, size_t ws_bytes, void* stream);
size_t ef_gqa_decode_workspace_bytes(int B, int Hq, int Hkv, int L, int D);

/* ---- Program 3c: decode attention over a sliding window with attention sinks -----------------
 * The single query sits at position L - 1 and sees keys j >= L - window plus the first `sinks`
 * keys (Section 7.3: sliding-window GQA; attention sinks -- only the chunks that cover the sink
 * tokens and the most recent `window` tokens are visited, the masked middle is skipped, and both
 * ranges contribute to one online reduction so they share one softmax normalisation).
 *   Q [B,Hq,D], K,V [B,Hkv,L,D] -> O [B,Hq,D].  window == 0 or window >= L: no window (sinks
 *   ignored) = ef_gqa_decode.  Supported shapes, workspace and errors as ef_gqa_decode. */
ef_status ef_gqa_decode_window(const void* Q, const void* K, const void* V, void* O,
                               int B, int Hq, int Hkv, int L, int D, float scale, int window, int sinks,
                               void* ws, size_t ws_bytes, void* stream);

/* ---- Program 3b: decode attention with per-sequence key lengths -----------------------------
 * The same rolling reducer over a batch whose sequences have different lengths (the serving
 * case behind the decode workloads of Section 7.1, batch sizes 1/8/16): batch entry b attends
 * keys [0, seq_lens[b]) of its K/V rows.  The chunks of all (batch, kv head) units still form
 * one list cut into equal contiguous ranges (Section 6.1 thread-block mapping; Section 4.4
 * Collection for units that span blocks), so a short sequence costs only its own bytes.
 *   Q [B,Hq,D], K,V [B,Hkv,Lmax,D] (rows at and beyond seq_lens[b] are padding: never used,
 *   may hold anything including NaN), seq_lens [B] int32 DEVICE pointer -> O [B,Hq,D].
 *   seq_lens[b] is clamped to [0, Lmax]; an entry with no keys gets O[b] = 0.
 * Supported: D == 128, Hq % Hkv == 0, Hq/Hkv <= 8, B <= 1024.
 * Workspace: ef_gqa_decode_workspace_bytes(B, Hq, Hkv, Lmax, D). */
ef_status ef_gqa_decode_varlen(const void* Q, const void* K, const void* V, const void* seq_lens, void* O,
                               int B, int Hq, int Hkv, int Lmax, int D, float scale,
                               void* ws, size_t ws_bytes, void* stream);

/* ---- Program 4: QK-normalised (causal) prefill attention ---------------------------------
 * qh = q * rsqrt(mean_d q^2 + eps) * gamma_q, kh likewise with gamma_k (over head_dim);
 * s_ij = scale * qh_i . kh_j for j <= i when causal != 0 (all j otherwise); softmax over j;
 * O = P @ V.  Definition: M0 -> M2 of Figure 4 with RMSNorm on Q and K; the inverse-RMS
 * factors are invariant along the contraction and move onto the logits (Table 1, factor
 * motion; Section 7.3, QK-normalized MLA).  Score and probability matrices never reach HBM
 * (Section 7.2, "Attention").
 *   Q,K,V [B,H,S,D], gamma_q [D], gamma_k [D] -> O [B,H,S,D].
 * Supported: D == 128, S >= 1, scale > 0. */
ef_status ef_qknorm_attn(const void* Q, const void* K, const void* V,
                         const void* gamma_q, const void* gamma_k, void* O,
                         int B, int H, int S, int D, float eps, float scale, int causal,
                         void* ws, size_t ws_bytes, void* stream);
size_t ef_qknorm_attn_workspace_bytes(int B, int H, int S, int D);

/* ---- Program 4b: the same attention with grouped KV heads, a sliding window and attention sinks ----
 * Mask variants of Section 7.3 (sliding-window attention with sink tokens: the first `sinks` keys plus
 * the last `window` keys of every query stay visible; key tiles in between are skipped, and the tiles of
 * both visible ranges feed ONE rolling softmax reduction) and grouped-query heads in prefill
 * (consecutive query heads share a K/V head).  With causal != 0:
 *   key j is visible to query i  iff  j <= i and (window == 0 or j > i - window or j < sinks).
 *   Q,O [B,Hq,S,D], K,V [B,Hkv,S,D], gamma_q/gamma_k [D].
 * Supported: D == 128, Hq % Hkv == 0, scale > 0; window > 0 and sinks > 0 need causal != 0; sinks <= 128;
 * sinks > 0 needs window > 0.  window >= S means no window.  ef_qknorm_attn is the case Hq == Hkv,
 * window == 0, sinks == 0.  Workspace: ef_qknorm_attn_workspace_bytes(B, Hkv, S, D). */
ef_status ef_qknorm_attn_ex(const void* Q, const void* K, const void* V,
                            const void* gamma_q, const void* gamma_k, void* O,
                            int B, int Hq, int Hkv, int S, int D, float eps, float scale, int causal,
                            int window, int sinks, void* ws, size_t ws_bytes, void* stream);

/* ---- Program 5: LoRA-fused linear ---------------------------------------------------------
 * Y = X @ W + alpha * (X @ A) @ Bm.
 * Definition: the LoRA workload (Section 7.1; Figure 2 factoring; Table 1 MatMul
 * reassociation).  Executed in the two-kernel form the paper's search selects (Section 7.2):
 * T = alpha * (X @ A) is stored once, then Y = [X | T] @ [W ; Bm] adds the rank-R update as
 * one extra K slab of the main contraction.
 *   X [M,K], W [K,N], A [K,R], Bm [R,N] -> Y [M,N].
 * Supported: R == 16, K % 64 == 0, N % 8 == 0. */
ef_status ef_lora_linear(const void* X, const void* W, const void* A, const void* Bm, void* Y,
                         int M, int K, int N, int R, float alpha,
                         void* ws, size_t ws_bytes, void* stream);
size_t ef_lora_linear_workspace_bytes(int M, int K, int N, int R);

/* ---- Decode attention without a caller workspace ---------------------------------------------
 * (The paper has no counterpart: this is a deployment convenience of the library.)
 * Same computation, arguments and supported shapes as ef_gqa_decode, for callers that are not
 * allowed to allocate device memory at the point of the call -- for example code that runs
 * inside a memory pool it must not grow, inside a real-time loop, or under a framework that
 * forbids cudaMalloc after start-up.  Instead of a caller workspace the call uses a scratch
 * array of 2,228,224 bytes that is part of the library image; every GPU that loads the library
 * holds that array until the process exits.
 *   - Limit: B * Hkv <= ef_gqa_decode_static_max_units() (1024); larger problems return
 *     EF_ERR_WORKSPACE and nothing is enqueued.  Other errors as for ef_gqa_decode.
 *   - The call allocates nothing (no cudaMalloc/cudaFree, no allocating library routine).  It
 *     enqueues one small memset (the status word and the arrival counters must start at zero,
 *     and the array keeps the previous call's contents) and then the decode kernel.
 *   - The FIRST call on each device looks up the array's device address (with that device
 *     current) and caches it; make that first call outside any stream capture.
 *   - All calls on a device share the one array: two calls that may overlap on the GPU (different
 *     streams, or graph branches) race on it.  Serialise them, or use ef_gqa_decode with separate
 *     workspaces. */
ef_status ef_gqa_decode_static(const void* Q, const void* K, const void* V, void* O,
                               int B, int Hq, int Hkv, int L, int D, float scale, void* stream);
size_t ef_gqa_decode_static_max_units(void);

/* ---- Workspace and status -------------------------------------------------------------------
 * (No counterpart in the paper: library plumbing.)
 * ef_workspace_init: enqueue zero-fill of the first min(ws_bytes, 64 KiB) bytes of ws on
 *   `stream` (status word, cross-block arrival counters).  Call once per workspace, again after
 *   ef_check_status reported EF_ERR_DEVICE_TIMEOUT, and before handing the workspace to a
 *   DIFFERENT entry point (each entry point keeps its own words in that window).  Calls of one
 *   entry point with different shapes may share a workspace that is large enough for each of them
 *   (the layout does not depend on the shape); calls that may overlap in time need separate ones.
 * ef_check_status: synchronise `stream`, read the 4-byte status word at ws[0]; returns EF_OK,
 *   EF_ERR_DEVICE_TIMEOUT, or EF_ERR_CUDA if the stream itself failed. */
ef_status ef_workspace_init(void* ws, size_t ws_bytes, void* stream);
ef_status ef_check_status(const void* ws, void* stream);

const char* ef_status_string(ef_status s);
int ef_last_cuda_error(void); /* last cudaError_t / CUresult seen by this thread's failing call */
int ef_version(void);

#ifdef __cplusplus
}
#endif
#endif /* EQUIFORGE_H_ */
