/*
 * tvm_attn.h -- C ABI of the fused attention + Jacobian-vector-product library for NVIDIA B200
 * (sm_100a).
 *
 * The operation is the one the Terminal Velocity Matching paper describes in Sec. 4 ("Flash
 * Attention JVP with backward pass") and App. C ("Flash Attention JVP with Backward Pass"):
 * scaled-dot-product attention that carries tangents next to the primal, and a backward pass that
 * differentiates through both outputs.
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers on the current device, owned by the caller, 16-byte
 *     aligned, (B, H, rows, d) with d contiguous: packed by default, with the strides given in
 *     tvm_attn_params otherwise.  Row statistics are packed (B, H, M) float.  The library never
 *     allocates, frees or keeps device memory.
 *   - Outputs are fully overwritten, never accumulated into.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = default stream)
 *     and the call returns without synchronising.  The forward and backward calls neither allocate
 *     nor synchronise, so they may be recorded into a CUDA graph by stream capture (make one call
 *     per device outside capture first: it loads the kernels); tvm_attn_check_status synchronises
 *     and the timing aid records events, so neither belongs inside a capture.
 *   - Return value: TVM_ATTN_OK or a negative tvm_attn_status.  No exception or abort crosses
 *     this boundary.  Concurrent calls from several host threads on different streams are allowed
 *     (each call with its own workspace); the per-kernel timing aid below is the exception and is to
 *     be driven from one thread while it is enabled.
 *   - After a call returns, its results are complete for any work enqueued later on the same stream
 *     (plain stream order), although the kernels of one backward call overlap one another.
 *   - Non-causal, no mask, bias or dropout: M queries attend to N keys per head (M = N by default).
 */
#ifndef TVM_ATTN_H_
#define TVM_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TVM_ATTN_OK = 0,
    TVM_ATTN_INVALID_ARG = -1,         /* null pointer, non-positive dim, misaligned pointer, bad dtype/flags */
    TVM_ATTN_UNSUPPORTED = -2,         /* d > 128 or d % 8 != 0, device is not sm_100, too many tiles  */
    TVM_ATTN_WORKSPACE_TOO_SMALL = -3, /* workspace_bytes < tvm_attn_jvp_workspace_bytes(...) */
    TVM_ATTN_CUDA_ERROR = -4,          /* a CUDA runtime/driver call or a launch failed */
    TVM_ATTN_DEVICE_TIMEOUT = -5,      /* a bounded on-device wait ran out (see tvm_attn_check_status) */
    TVM_ATTN_TOO_LARGE = -6            /* B*H*N exceeds the built-in scratch of tvm_attn_jvp_bwd_noalloc */
} tvm_attn_status;

/* dtype of the eight/sixteen (B,H,N,d) tensors */
#define TVM_ATTN_BF16 0 /* bf16 tensors, fp32 accumulation, tensor-core kernels (the hot path)      */
#define TVM_ATTN_FP32 1 /* fp32 tensors, fp32 CUDA-core kernels (validation mode, not a fast path)  */

/* flags */
#define TVM_ATTN_FLAG_CUDA_CORES 1u /* run the CUDA-core validation kernels also for bf16 tensors   */

typedef struct {
    int32_t B, H, N, d; /* batch, heads, keys per head, head dim; 8 <= d <= 128, d % 8 == 0          */
    float scale;        /* softmax scale alpha of App. C; 0.0f selects 1/sqrt(d) with the true d     */
    int32_t dtype;      /* TVM_ATTN_BF16 or TVM_ATTN_FP32                                            */
    uint32_t flags;     /* 0 or TVM_ATTN_FLAG_*                                                      */
    int32_t M;          /* queries per head (App. C "Background": Q in R^{M x d}, K, V in R^{N x d});
                           0 = N, self-attention                                                      */
    /* Element strides {row, head, batch} of the query-side tensors (Q, tQ, O, tO, dO, dtO, dQ, dtQ: M rows per
       head) and of the key-side tensors (K, V, tK, tV, dK, dV, dtK, dtV: N rows per head).  All three zero selects
       the packed layouts (B, H, M, d) and (B, H, N, d).  A (B, rows, H, d) tensor, or the Q, K, V slices of a
       fused (B, rows, 3, H, d) projection read and written in place, are {row = H*d or 3*H*d, head = d,
       batch = rows * row}.  The d elements of a row are contiguous; every stride is a multiple of 8 elements;
       row >= d.  The statistics lse, mu and the workspace are always packed (B, H, M).  Strides and M != N
       need d <= 80 (TVM_ATTN_UNSUPPORTED above). */
    int64_t q_strides[3];
    int64_t k_strides[3];
} tvm_attn_params;

/*
 * Bytes of device scratch the forward (is_bwd == 0) or backward (is_bwd != 0) call needs for these
 * parameters.  The forward needs none.  The backward keeps three floats per query row there (the row
 * sums of App. C "Step 1", in the form rowsum(dtO*O) and rowsum(dO*O) + rowsum(dtO*tO), and lse in
 * log2 units).
 * Returns 0 for invalid parameters.
 */
size_t tvm_attn_jvp_workspace_bytes(const tvm_attn_params* p, int is_bwd);

/*
 * Forward (paper Sec. 4 item (i); App. C Eq. "sdpa" and the definitions of P, S, N, S-dot, mu
 * under "Step 1"; "Caching softmax statistics").  Per head, with A = alpha Q K^T, P = softmax_rows(A),
 * T = alpha (tQ K^T + Q tK^T), mu = rowsum(P*T):
 *     O  = P V                      tO = (P * (T - mu)) V + P tV
 *     lse = log rowsum(exp(A))      (natural log, of the SCALED scores)
 * computed with an online softmax; no N x N matrix is written to memory.
 *   in : Q, K, V, tQ, tK, tV   (B,H,N,d) dtype
 *   out: O, tO                 (B,H,N,d) dtype, rounded to nearest even from fp32
 *        lse, mu               (B,H,N) float; the statistics the backward needs (normalised mu, so
 *                              the separate row sum l of App. C is not stored)
 *   workspace: may be NULL (workspace_bytes 0).
 */
int tvm_attn_jvp_fwd(const tvm_attn_params* p, const void* Q, const void* K, const void* V,
                     const void* tQ, const void* tK, const void* tV, void* O, void* tO, float* lse,
                     float* mu, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Backward through both outputs (paper Sec. 4 item (iii); App. C "Multi-step backward pass",
 * steps 1-6, plus the standard attention backward for dO that the paper sums in).  With
 * G = dO, Hc = dtO, Nn = T - mu, D = Hc V^T, X = G V^T + Hc tV^T,
 * W = P * (D - Sigma_1), dA = P * (X - rowsum(G*O) - Sigma_2) + W * Nn:
 *     dV = P^T G + (P*Nn)^T Hc     dtV = P^T Hc
 *     dQ = alpha (dA K + W tK)     dtQ = alpha W K
 *     dK = alpha (dA^T Q + W^T tQ) dtK = alpha W^T Q
 *   in : Q, K, V, tQ, tK, tV and the forward's O, tO, lse, mu; dO, dtO (B,H,N,d) dtype.
 *        One of dO, dtO may be NULL and then counts as zero; it is never read and the work that only
 *        it feeds is skipped.  dtO == NULL is the "detach JVP" setting of Sec. 5.3 (memory and runtime
 *        table: no gradient flows through tO): what remains is the standard attention backward for dO.
 *        dO == NULL leaves steps 1-6 of App. C alone.  Both NULL is TVM_ATTN_INVALID_ARG.  For
 *        d > 80 both cotangents are required (TVM_ATTN_UNSUPPORTED otherwise).
 *   out: dQ, dK, dV, dtQ, dtK, dtV (B,H,N,d) dtype.  With dtO == NULL the tangent gradients are
 *        identically zero: dtQ, dtK, dtV may then be NULL, and those given are set to zero.
 *   workspace: device scratch of at least tvm_attn_jvp_workspace_bytes(p, 1) bytes, 16-byte
 *        aligned; contents on return are unspecified.  Calls sharing one workspace must not
 *        overlap on the device.
 */
int tvm_attn_jvp_bwd(const tvm_attn_params* p, const void* Q, const void* K, const void* V,
                     const void* tQ, const void* tK, const void* tV, const void* O, const void* tO,
                     const float* lse, const float* mu, const void* dO, const void* dtO, void* dQ,
                     void* dK, void* dV, void* dtQ, void* dtK, void* dtV, void* workspace,
                     size_t workspace_bytes, void* cuda_stream);

/*
 * Backward pass for callers that cannot allocate device memory (no counterpart in the paper).
 *
 * Some hosts of this library may not call cudaMalloc at the point where they need the backward: code
 * running inside another framework's memory plan with every byte already assigned, a real-time or
 * embedded loop where an allocation could fail or stall, a plug-in that is handed tensors but no
 * allocator.  tvm_attn_jvp_bwd asks them for a workspace they have no way to provide.  This entry
 * point computes exactly what tvm_attn_jvp_bwd computes, with the same arguments minus the workspace,
 * and keeps its scratch in a fixed array inside the library's device image instead.
 *
 *   - Limit: B * H * N <= TVM_ATTN_NOALLOC_MAX_ROWS.  Larger problems return TVM_ATTN_TOO_LARGE before
 *     anything is launched; use tvm_attn_jvp_bwd with your own workspace for those.
 *   - Cost: the array (12 bytes per row, 3 MiB) is part of the library image, so every GPU that loads the
 *     library holds it until the process exits, whether or not this function is ever called.
 *   - It calls neither cudaMalloc nor cudaFree nor any allocating library routine.
 *   - The first call on each device looks up the array's device address (once per device, with that
 *     device current) and keeps it for the life of the process.  Make that first call outside any
 *     stream capture.  Devices with index 0..63 are supported (TVM_ATTN_CUDA_ERROR beyond), and the
 *     kept address does not survive a cudaDeviceReset of that device.
 *   - All calls on a device share the one array.  Nothing in it has to start at zero (the pass rewrites
 *     all of it before reading it) and its contents after a call are unspecified.  Two calls that may
 *     run at the same time on the GPU (different streams, different host threads) race on it: serialise
 *     them, or give the concurrent ones their own workspace through tvm_attn_jvp_bwd.
 */
#define TVM_ATTN_NOALLOC_MAX_ROWS 262144
int tvm_attn_jvp_bwd_noalloc(const tvm_attn_params* p, const void* Q, const void* K, const void* V,
                             const void* tQ, const void* tK, const void* tV, const void* O, const void* tO,
                             const float* lse, const float* mu, const void* dO, const void* dtO, void* dQ,
                             void* dK, void* dV, void* dtQ, void* dtK, void* dtV, void* cuda_stream);

/*
 * RMSNorm QK-normalisation with a tangent: the step in front of the attention in the paper's transformer
 * (Sec. 4 "semi-Lipschitz control": RMSNorm as QK-norm with a learnable scale; App. "Lipschitzness of
 * RMSNorm" gives the definition and the Jacobian).  Per row x of Q (and of K), with the row's tangent tx and
 * a per-channel scale g of d floats shared by all rows:
 *     r = sqrt(mean(x^2) + eps)      y = g * x / r      ty = g * (tx / r - x (x . tx) / (d r^3))
 * (the paper prints the sum under the root without the square; its Jacobian is that of the squared form,
 * which is what is computed).  One call normalises Q and K; its outputs are the Q, tQ, K, tK of
 * tvm_attn_jvp_fwd.  Memory-bound streaming kernels: every tensor is read or written once.
 *   in : Q, tQ, K, tK (B,H,N,d) dtype; gQ, gK: d floats each (device, 16-byte aligned); eps >= 0
 *   out: Qn, tQn, Kn, tKn (B,H,N,d) dtype
 */
int tvm_qk_rmsnorm_jvp_fwd(const tvm_attn_params* p, float eps, const void* Q, const void* tQ, const void* K,
                           const void* tK, const float* gQ, const float* gK, void* Qn, void* tQn, void* Kn,
                           void* tKn, void* cuda_stream);

/*
 * Backward of tvm_qk_rmsnorm_jvp_fwd through both outputs: given the cotangents of Qn, tQn, Kn, tKn (what
 * tvm_attn_jvp_bwd returns as dQ, dtQ, dK, dtK), the gradients of the un-normalised Q, tQ, K, tK and of the
 * two scales.  With J = (I - u u^T / d) / r, u = x / r (the Jacobian of App. "Lipschitzness of RMSNorm"),
 * a = g * dy, b = g * dty:
 *     dtx = J b        dx = J a + d/dx [ b . (J(x) tx) ]        dg = sum over rows of dy * u + dty * (J tx)
 * The normalised tensors are not needed: r is recomputed from x.  dgQ, dgK (d floats each) are written, not
 * accumulated into, and are bit-reproducible (fixed summation order).
 *   workspace: at least tvm_qk_rmsnorm_jvp_workspace_bytes(p) bytes of device scratch, 16-byte aligned
 *        (partial sums of the scale gradients); 0 is returned for invalid parameters.
 */
size_t tvm_qk_rmsnorm_jvp_workspace_bytes(const tvm_attn_params* p);
int tvm_qk_rmsnorm_jvp_bwd(const tvm_attn_params* p, float eps, const void* Q, const void* tQ, const void* K,
                           const void* tK, const float* gQ, const float* gK, const void* dQn, const void* dtQn,
                           const void* dKn, const void* dtKn, void* dQ, void* dtQ, void* dK, void* dtK,
                           float* dgQ, float* dgK, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Synchronises `cuda_stream` and reports what the kernels enqueued so far on the current device
 * recorded: TVM_ATTN_OK, TVM_ATTN_DEVICE_TIMEOUT if a bounded wait inside a tensor-core kernel gave
 * up (its outputs are then unspecified; the context stays usable), or TVM_ATTN_CUDA_ERROR.  Clears
 * the recorded status.  (No counterpart in the paper: error reporting of this library.)
 * The status is one word per device, not per stream: tensor-core kernels that start while it is raised
 * return at once without touching their outputs, and with several host threads the time-out reported
 * to one of them may have been raised by another thread's call.
 */
int tvm_attn_check_status(void* cuda_stream);

/*
 * Exercises the time-out reporting without disturbing a real kernel (no counterpart in the paper).
 * Enqueues a one-warp kernel that waits on a barrier nobody signals, with the same bounded wait the
 * tensor-core kernels use, and gives up after `limit_ns` nanoseconds (1 .. 100,000,000; a millisecond
 * is plenty).  It then raises the device status exactly like a kernel whose wait ran out: the next
 * tvm_attn_check_status returns TVM_ATTN_DEVICE_TIMEOUT, and tensor-core kernels enqueued in between
 * are no-ops.  Nothing hangs and the context stays usable.
 */
int tvm_attn_selftest_timeout(uint64_t limit_ns, void* cuda_stream);

/*
 * Per-kernel timing aid (no counterpart in the paper).  While enabled, tvm_attn_jvp_fwd/bwd record
 * CUDA events on the caller's stream around every kernel they launch.  tvm_attn_get_profile waits
 * for the most recent profiled call and writes the duration in milliseconds of each of its kernels
 * to ms[0..], in launch order (forward: 1 kernel; backward: row sums, dV/dtV, dK/dtK, dQ/dtQ), and
 * returns how many it wrote (at most `capacity`), or a negative status.  Process-wide state: use
 * from one host thread at a time.  Creates CUDA events, no device memory.
 */
int tvm_attn_set_profiling(int enable);
int tvm_attn_get_profile(float* ms, int capacity);

/* Number of this library's kernels launched by the calling process so far (all threads). */
uint64_t tvm_attn_launch_count(void);

/* Static, human-readable text for a status code. */
const char* tvm_attn_strerror(int code);

/* Library version: major * 10000 + minor * 100 + patch. */
int tvm_attn_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TVM_ATTN_H_ */
