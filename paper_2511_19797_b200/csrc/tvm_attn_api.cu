// C-ABI entry points of the attention-JVP library (see include/tvm_attn.h): argument checks, TMA
// tensor-map construction and kernel launches.  No device memory is allocated here.
#include "tvm_attn.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>

#include "dual_attn_sm100.cuh"
#include "jvp_bwd_sm100.cuh"
#include "jvp_fwd_sm100.cuh"
#include "qk_rmsnorm.cuh"
#include "simt_kernels.cuh"

namespace tvm_attn {

static std::atomic<uint64_t> g_launches{0};

// Number of SMs of the current device (a fact of the hardware: looked up once per device index); <= 0 on error.
static int device_sm_count() {
    static std::atomic<int> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return -1;
    if (dev < 64) {
        const int v = cached[dev].load(std::memory_order_relaxed);
        if (v > 0) return v;
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return -1;
    if (dev < 64) cached[dev].store(sms, std::memory_order_relaxed);
    return sms;
}
__device__ int g_status_word = 0;  // raised by a tensor-core kernel whose bounded wait ran out

// Optional per-kernel timing: events recorded around each launch of the most recent call.  While it is
// disabled (the normal state) a call only reads the atomic flag, so concurrent calls from several host
// threads do not touch shared state; while it is enabled the library is to be driven by one thread.
struct Profiler {
    std::atomic<bool> enabled{false};
    std::atomic<int> count{0};  // kernels recorded by the last call
    cudaEvent_t ev[8] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    void begin_call() { if (enabled.load(std::memory_order_relaxed)) count.store(0); }
    void mark(cudaStream_t st, int idx) {
        if (idx >= 8) return;
        if (!ev[idx] && cudaEventCreate(&ev[idx]) != cudaSuccess) { ev[idx] = nullptr; return; }
        cudaEventRecord(ev[idx], st);
    }
    void before(cudaStream_t st) { if (enabled.load(std::memory_order_relaxed) && count.load() == 0) mark(st, 0); }
    void after(cudaStream_t st) { if (enabled.load(std::memory_order_relaxed)) { mark(st, count.load() + 1); count.fetch_add(1); } }
};
static Profiler g_prof;

struct Shape {
    int B, H, N, M, d, dp;   // N keys, M queries per head
    long long BH;
    float alpha;
    bool fp32, simt;
    Geom q, k;               // query side (M rows) and key side (N rows)
    bool plain;              // self-attention on packed (B, H, N, d) tensors
};

// Strides of one side: all zero selects the packed (B, H, rows, d) layout.
static int side_geometry(const int64_t st[3], int rows, int H, int d, Geom* g) {
    g->rows = rows;
    if (st[0] == 0 && st[1] == 0 && st[2] == 0) {
        g->rs = d; g->hs = (long long)rows * d; g->bs = (long long)H * rows * d;
        return TVM_ATTN_OK;
    }
    // rows must not overlap inside themselves and every row must start on a 16-byte boundary (TMA, vector loads)
    if (st[0] < d || st[1] <= 0 || st[2] <= 0 || st[0] % 8 || st[1] % 8 || st[2] % 8) return TVM_ATTN_INVALID_ARG;
    if (st[0] > (1LL << 36) || st[1] > (1LL << 36) || st[2] > (1LL << 36)) return TVM_ATTN_UNSUPPORTED;  // TMA strides < 2^40 bytes
    g->rs = st[0]; g->hs = st[1]; g->bs = st[2];
    return TVM_ATTN_OK;
}

static int check_params(const tvm_attn_params* p, Shape* s) {
    if (!p) return TVM_ATTN_INVALID_ARG;
    if (p->B <= 0 || p->H <= 0 || p->N <= 0 || p->d <= 0 || p->M < 0) return TVM_ATTN_INVALID_ARG;
    if (p->dtype != TVM_ATTN_BF16 && p->dtype != TVM_ATTN_FP32) return TVM_ATTN_INVALID_ARG;
    if (p->flags & ~TVM_ATTN_FLAG_CUDA_CORES) return TVM_ATTN_INVALID_ARG;
    if (!(p->scale >= 0.0f) || !std::isfinite(p->scale)) return TVM_ATTN_INVALID_ARG;
    if (p->d > 128 || p->d % 8 != 0) return TVM_ATTN_UNSUPPORTED;
    s->B = p->B; s->H = p->H; s->N = p->N; s->d = p->d;
    s->M = p->M > 0 ? p->M : p->N;
    int rg = side_geometry(p->q_strides, s->M, p->H, p->d, &s->q);
    if (rg != TVM_ATTN_OK) return rg;
    rg = side_geometry(p->k_strides, s->N, p->H, p->d, &s->k);
    if (rg != TVM_ATTN_OK) return rg;
    s->plain = s->M == s->N && s->q.rs == s->d && s->k.rs == s->d && s->q.hs == (long long)s->N * s->d && s->k.hs == s->q.hs &&
               s->q.bs == (long long)s->H * s->N * s->d && s->k.bs == s->q.bs;
    s->dp = (p->d + 15) / 16 * 16;
    s->BH = (long long)p->B * p->H;
    s->alpha = p->scale == 0.0f ? 1.0f / std::sqrt((float)p->d) : p->scale;
    s->fp32 = p->dtype == TVM_ATTN_FP32;
    s->simt = s->fp32 || (p->flags & TVM_ATTN_FLAG_CUDA_CORES);
    // every kernel flattens (head, row tile) into blockIdx.x
    const long long longer = s->M > s->N ? s->M : s->N;
    const long long tiles16 = (longer + 15LL) / 16;
    if (s->BH * tiles16 > 2147483647LL) return TVM_ATTN_UNSUPPORTED;
    if (s->BH > 2147483647LL / longer) return TVM_ATTN_UNSUPPORTED;  // B*H*rows indexable as int
    return TVM_ATTN_OK;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int cuda_status(cudaError_t e) { return e == cudaSuccess ? TVM_ATTN_OK : TVM_ATTN_CUDA_ERROR; }

// ------------------------------------------------------------------------------------------------
// CUDA-core path
template <typename T>
static int simt_fwd(const Shape& s, const void* Q, const void* K, const void* V, const void* tQ, const void* tK,
                    const void* tV, void* O, void* tO, float* lse, float* mu, cudaStream_t st) {
    const size_t smem = simt_smem_bytes(s.d, 2);
    cudaError_t e = cudaFuncSetAttribute(simt_fwd_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return TVM_ATTN_CUDA_ERROR;
    const unsigned grid = (unsigned)(s.BH * ((s.M + SIMT_ROWS - 1) / SIMT_ROWS));
    g_prof.before(st);
    simt_fwd_kernel<T><<<grid, SIMT_THREADS, smem, st>>>((const T*)Q, (const T*)K, (const T*)V, (const T*)tQ,
                                                         (const T*)tK, (const T*)tV, (T*)O, (T*)tO, lse, mu, s.q, s.k, s.H,
                                                         s.d, s.alpha);
    g_prof.after(st);
    g_launches += 1;
    return cuda_status(cudaGetLastError());
}

static bool q_packed(const Shape& s) {
    return s.q.rs == s.d && s.q.hs == (long long)s.M * s.d && s.q.bs == (long long)s.H * s.M * s.d;
}

template <typename T>
static int launch_rowsums(const Shape& s, const void* G, const void* Hc, const void* O, const void* tO, const float* lse,
                          float* sig1, float* cvec, float* lse2, cudaStream_t st) {
    const long long rows = s.BH * s.M;
    const int cpr = s.d * (int)sizeof(T) / 16;  // 16-byte chunks per row (d % 8 == 0)
    const int gs = cpr;                          // lanes per row
    if (gs > 32) return TVM_ATTN_UNSUPPORTED;   // d <= 128 keeps a row within one warp
    const long long rows_per_block = (long long)(ROWSUM_THREADS / 32) * ROWSUM_UNROLL * (32 / gs);
    const unsigned grid = (unsigned)((rows + rows_per_block - 1) / rows_per_block);
    g_prof.before(st);
    bwd_rowsums_kernel<T><<<grid, ROWSUM_THREADS, 0, st>>>((const T*)G, (const T*)Hc, (const T*)O, (const T*)tO, lse, sig1,
                                                           cvec, lse2, rows, s.q, q_packed(s) ? 0 : s.H, s.d, cpr, gs);
    g_prof.after(st);
    g_launches += 1;
    return cuda_status(cudaGetLastError());
}

template <typename T>
static int simt_bwd(const Shape& s, const void* Q, const void* K, const void* V, const void* tQ, const void* tK,
                    const void* tV, const float* lse, const float* mu, const void* G, const void* Hc,
                    const float* sig1, const float* cvec, void* dQ, void* dK, void* dV, void* dtQ, void* dtK, void* dtV,
                    cudaStream_t st) {
    const size_t smem = simt_smem_bytes(s.d, 4);
    if (cudaFuncSetAttribute(simt_bwd_dq_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaFuncSetAttribute(simt_bwd_dkv_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return TVM_ATTN_CUDA_ERROR;
    const unsigned grid_q = (unsigned)(s.BH * ((s.M + SIMT_ROWS - 1) / SIMT_ROWS));
    const unsigned grid_k = (unsigned)(s.BH * ((s.N + SIMT_ROWS - 1) / SIMT_ROWS));
    simt_bwd_dq_kernel<T><<<grid_q, SIMT_THREADS, smem, st>>>((const T*)Q, (const T*)K, (const T*)V, (const T*)tQ,
                                                              (const T*)tK, (const T*)tV, (const T*)G, (const T*)Hc, lse,
                                                              mu, sig1, cvec, (T*)dQ, (T*)dtQ, s.q, s.k, s.H, s.d, s.alpha);
    g_prof.after(st);
    simt_bwd_dkv_kernel<T><<<grid_k, SIMT_THREADS, smem, st>>>((const T*)Q, (const T*)K, (const T*)V, (const T*)tQ,
                                                               (const T*)tK, (const T*)tV, (const T*)G, (const T*)Hc,
                                                               lse, mu, sig1, cvec, (T*)dK, (T*)dV, (T*)dtK, (T*)dtV,
                                                               s.q, s.k, s.H, s.d, s.alpha);
    g_prof.after(st);
    g_launches += 2;
    return cuda_status(cudaGetLastError());
}

// ------------------------------------------------------------------------------------------------
// Tensor-core path
typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static encode_tiled_fn get_encode_fn() {
    static encode_tiled_fn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<encode_tiled_fn>(sym);
    });
    return fn;
}

// A bf16 tensor of one side viewed as a 4-D tensor (d, rows, H, B) with that side's strides; a box is 64 columns x
// `rows` rows of one head with the 128-byte swizzle; columns or rows beyond the tensor read as zero.
static int make_tmap(CUtensorMap* m, const void* ptr, const Shape& s, const Geom& g, int rows) {
    encode_tiled_fn fn = get_encode_fn();
    if (!fn) return TVM_ATTN_CUDA_ERROR;
    cuuint64_t dims[4] = {(cuuint64_t)s.d, (cuuint64_t)g.rows, (cuuint64_t)s.H, (cuuint64_t)s.B};
    cuuint64_t strides[3] = {(cuuint64_t)g.rs * 2, (cuuint64_t)g.hs * 2, (cuuint64_t)g.bs * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)rows, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? TVM_ATTN_OK : TVM_ATTN_CUDA_ERROR;
}

// Packed (B,H,N,d) bf16 viewed as a 3-D tensor (d, N, B*H): the kernels for head dims above 80.
static int make_tmap3(CUtensorMap* m, const void* ptr, const Shape& s, int rows) {
    encode_tiled_fn fn = get_encode_fn();
    if (!fn) return TVM_ATTN_CUDA_ERROR;
    cuuint64_t dims[3] = {(cuuint64_t)s.d, (cuuint64_t)s.N, (cuuint64_t)s.BH};
    cuuint64_t strides[2] = {(cuuint64_t)s.d * 2, (cuuint64_t)s.N * s.d * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? TVM_ATTN_OK : TVM_ATTN_CUDA_ERROR;
}

static int device_is_sm100() {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return TVM_ATTN_CUDA_ERROR;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return TVM_ATTN_CUDA_ERROR;
    return major == 10 ? TVM_ATTN_OK : TVM_ATTN_UNSUPPORTED;
}

static int* status_word_ptr() {
    int* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_status_word) != cudaSuccess) return nullptr;
    return ptr;
}

template <int MODE, int NA>
static int launch_tc(const Shape& s, const void* const own[4], const void* const strm[4], const TcParams& prm,
                     cudaStream_t st) {
    using C = TcCfg<MODE, NA>;
    CUtensorMap mo[4], ms[4];
    for (int t = 0; t < 4; ++t) {
        const void* po = own[t < C::NOWN ? t : 0];
        int rc = make_tmap3(&mo[t], po, s, TC_OWN_ROWS);
        if (rc != TVM_ATTN_OK) return rc;
        rc = make_tmap3(&ms[t], strm[t], s, C::BC);
        if (rc != TVM_ATTN_OK) return rc;
    }
    auto kern = dual_attn_kernel<MODE, NA>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) != cudaSuccess)
        return TVM_ATTN_CUDA_ERROR;
    const long long grid = s.BH * ((s.N + TC_OWN_ROWS - 1) / TC_OWN_ROWS);
    g_prof.before(st);
    kern<<<(unsigned)grid, TC_THREADS, C::SMEM_BYTES, st>>>(mo[0], mo[1], mo[2], mo[3], ms[0], ms[1], ms[2], ms[3], prm);
    g_prof.after(st);
    g_launches += 1;
    return cuda_status(cudaGetLastError());
}

template <int MODE>
static int launch_tc_na(const Shape& s, const void* const own[4], const void* const strm[4], const TcParams& prm,
                        cudaStream_t st) {
    return s.d <= 64 ? launch_tc<MODE, 1>(s, own, strm, prm, st) : launch_tc<MODE, 2>(s, own, strm, prm, st);
}

// Forward for padded head dims up to 80: operands Q, tQ live in tensor memory (jvp_fwd_sm100.cuh).
template <int DP>
static int launch_fwd(const Shape& s, const void* const strm[4], const FwdParams& prm, cudaStream_t st) {
    using C = FwdCfg<DP>;
    CUtensorMap m[4];
    for (int t = 0; t < 4; ++t) {
        const int rc = make_tmap(&m[t], strm[t], s, s.k, FWD_BC);
        if (rc != TVM_ATTN_OK) return rc;
    }
    auto kern = jvp_fwd_kernel<DP>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) != cudaSuccess)
        return TVM_ATTN_CUDA_ERROR;
    // one CTA per SM (each needs the whole tensor memory and most of the shared memory of one); the work
    // items go round-robin over them
    const long long items = s.BH * ((s.M + FWD_ROWS - 1) / FWD_ROWS);
    const int sms = device_sm_count();
    if (sms <= 0) return TVM_ATTN_CUDA_ERROR;
    const long long grid = items < sms ? items : sms;
    g_prof.before(st);
    kern<<<(unsigned)grid, FWD_THREADS, C::SMEM_BYTES, st>>>(m[0], m[1], m[2], m[3], prm);
    g_prof.after(st);
    g_launches += 1;
    return cuda_status(cudaGetLastError());
}

// One backward pass for padded head dims up to 80 (jvp_bwd_sm100.cuh).  own: X0..X3; strm: E ring (0, 1), L ring (2, 3).
template <int MODE, int DP>
static int launch_bwd_pass(const Shape& s, const void* const own[4], const void* const strm[4], BwdParams prm, cudaStream_t st) {
    using C = BwdCfg<MODE, DP>;
    CUtensorMap ms[4], mo[2];
    // DV, DK: keys own, queries stream; DQ: queries own, keys stream
    prm.o = MODE == BWD_DQ ? s.q : s.k;
    prm.s = MODE == BWD_DQ ? s.k : s.q;
    for (int t = 0; t < 4; ++t) {
        // an absent cotangent (null) is never loaded: its map is built on a present tensor and stays unused
        const int rc = make_tmap(&ms[t], strm[t] ? strm[t] : strm[t ^ 1], s, prm.s, C::BC);
        if (rc != TVM_ATTN_OK) return rc;
        prm.strm[t] = static_cast<const __nv_bfloat16*>(strm[t]);
        prm.own[t] = static_cast<const __nv_bfloat16*>(own[t]);
    }
    for (int t = 0; t < 2; ++t) {
        const int rc = make_tmap(&mo[t], own[C::NPAIR == 2 ? C::XS0 + t : t], s, prm.o, BWD_ROWS);  // never a cotangent
        if (rc != TVM_ATTN_OK) return rc;
    }
    // dtO absent: the specialisation that leaves the tangent path out (only instantiated for the padded head dims
    // 64 and 80 of the transformer shapes; other head dims run the general kernel, which skips what it can)
    constexpr bool HAS_HZ = DP == 64 || DP == 80;
    auto kern = (HAS_HZ && (prm.absent & ABSENT_HC)) ? jvp_bwd_kernel<MODE, DP, HAS_HZ> : jvp_bwd_kernel<MODE, DP, false>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) != cudaSuccess)
        return TVM_ATTN_CUDA_ERROR;
    // one CTA per SM (each needs the whole tensor memory and most of the shared memory of one); the work
    // items go round-robin over them
    const long long items = s.BH * ((prm.o.rows + BWD_ROWS - 1) / BWD_ROWS);
    const int sms = device_sm_count();
    if (sms <= 0) return TVM_ATTN_CUDA_ERROR;
    const long long grid = items < sms ? items : sms;
    g_prof.before(st);
    {
        // DK and DQ read nothing that the pass before them writes (DV, DK and DQ all depend on the row-sums
        // pre-pass only, which has completed before DV starts), so their CTAs may fill the SMs that the last,
        // partial wave of the pass before leaves idle: programmatic dependent launch, with every CTA of these
        // kernels releasing its dependents at once.  None waits for its primary before it works; each waits for
        // it once at the very end (griddepcontrol.wait in the teardown), so that DQ cannot complete before DK, nor
        // DK before DV: work enqueued behind the call still sees all six gradients.  Not while per-kernel events
        // are being recorded: they would time overlapping kernels.
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)grid);
        cfg.blockDim = dim3(BWD_THREADS);
        cfg.dynamicSmemBytes = C::SMEM_BYTES;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = (MODE != BWD_DV && !g_prof.enabled.load(std::memory_order_relaxed)) ? 1 : 0;
        if (cudaLaunchKernelEx(&cfg, kern, ms[0], ms[1], ms[2], ms[3], mo[0], mo[1], prm) != cudaSuccess)
            return cuda_status(cudaGetLastError());
    }
    g_prof.after(st);
    g_launches += 1;
    return cuda_status(cudaGetLastError());
}

template <int MODE>
static int launch_bwd_pass_dp(const Shape& s, const void* const own[4], const void* const strm[4], const BwdParams& prm,
                              cudaStream_t st) {
    switch (s.dp) {
        case 16: return launch_bwd_pass<MODE, 16>(s, own, strm, prm, st);
        case 32: return launch_bwd_pass<MODE, 32>(s, own, strm, prm, st);
        case 48: return launch_bwd_pass<MODE, 48>(s, own, strm, prm, st);
        case 64: return launch_bwd_pass<MODE, 64>(s, own, strm, prm, st);
        default: return launch_bwd_pass<MODE, 80>(s, own, strm, prm, st);
    }
}

static TcParams base_params(const Shape& s, int* status) {
    TcParams prm;
    std::memset(&prm, 0, sizeof prm);
    prm.N = s.N; prm.d = s.d; prm.dp = s.dp; prm.BH = (int)s.BH;
    prm.alpha = s.alpha;
    prm.c2 = s.alpha * 1.4426950408889634f;
    prm.out_scale = 1.0f;
    prm.status = status;
    return prm;
}

// Scratch of tvm_attn_jvp_bwd_noalloc: three floats per row, for callers that cannot allocate.  In host code
// this name is only a handle for cudaGetSymbolAddress, never a device pointer.
static __device__ __align__(256) float g_noalloc_scratch[3 * TVM_ATTN_NOALLOC_MAX_ROWS];
static constexpr int kMaxDevices = 64;
static float* g_noalloc_addr[kMaxDevices] = {};  // device address of the array, per device
static std::mutex g_noalloc_mutex;

// Device address of the scratch array on the current device, looked up on first use.
static int noalloc_scratch_address(float** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TVM_ATTN_CUDA_ERROR;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_addr[dev]) {
        float* ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_scratch) != cudaSuccess || !ptr)
            return TVM_ATTN_CUDA_ERROR;
        g_noalloc_addr[dev] = ptr;
    }
    *out = g_noalloc_addr[dev];
    return TVM_ATTN_OK;
}

// One warp waits, with a limit, on an mbarrier that nobody arrives at: the same bounded wait the tensor-core
// kernels use, made to run out on purpose so that the time-out reporting can be exercised without disturbing
// a real kernel.  Raises the device status word like they do.
__global__ void selftest_timeout_kernel(int* status, unsigned long long limit_ns) {
    __shared__ __align__(8) unsigned long long barrier;
    __shared__ int abort_flag;
    if (*reinterpret_cast<volatile int*>(status) != 0) return;
    const uint32_t bar = ptx::smem_u32(&barrier);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        ptx::mbar_init(bar, 1);
        ptx::fence_mbar_init();
    }
    __syncwarp();
    const bool ok = ptx::mbar_wait_warp(bar, 0, &abort_flag, limit_ns);
    if (!ok && threadIdx.x == 0 && abort_flag) atomicExch(status, 1);
}

// ------------------------------------------------------------------------------------------------
// RMSNorm QK-normalisation prologue
static int rms_geometry(const Shape& s, int* cpr, int* gs) {
    *cpr = s.d * (s.fp32 ? 4 : 2) / 16;
    *gs = *cpr;   // lanes per row
    return *gs <= 32 ? TVM_ATTN_OK : TVM_ATTN_UNSUPPORTED;
}

template <typename T>
static int rms_fwd(const Shape& s, float eps, const void* Q, const void* tQ, const void* K, const void* tK, const float* gQ,
                   const float* gK, void* Qn, void* tQn, void* Kn, void* tKn, cudaStream_t st) {
    int cpr, gs;
    const int rc = rms_geometry(s, &cpr, &gs);
    if (rc != TVM_ATTN_OK) return rc;
    const long long rows_q = s.BH * s.M, rows_k = s.BH * s.N, rows_per_block = (long long)(RMS_THREADS / 32) * (32 / gs);
    const RmsFwdSide<T> q{(const T*)Q, (const T*)tQ, gQ, (T*)Qn, (T*)tQn, s.q, rows_q};
    const RmsFwdSide<T> k{(const T*)K, (const T*)tK, gK, (T*)Kn, (T*)tKn, s.k, rows_k};
    const long long rows = rows_q > rows_k ? rows_q : rows_k;
    const dim3 grid((unsigned)((rows + rows_per_block - 1) / rows_per_block), 2);
    qk_rmsnorm_jvp_fwd_kernel<T><<<grid, RMS_THREADS, 0, st>>>(q, k, s.H, s.d, cpr, gs, eps);
    g_launches += 1;
    return cuda_status(cudaGetLastError());
}

template <typename T>
static int rms_bwd(const Shape& s, float eps, const void* Q, const void* tQ, const void* K, const void* tK, const float* gQ,
                   const float* gK, const void* dQn, const void* dtQn, const void* dKn, const void* dtKn, void* dQ, void* dtQ,
                   void* dK, void* dtK, float* dgQ, float* dgK, float* partial, cudaStream_t st) {
    int cpr, gs;
    const int rc = rms_geometry(s, &cpr, &gs);
    if (rc != TVM_ATTN_OK) return rc;
    float* pq = partial;
    float* pk = partial + (size_t)RMS_BWD_BLOCKS * s.d;
    const RmsBwdSide<T> q{(const T*)Q, (const T*)tQ, gQ, (const T*)dQn, (const T*)dtQn, (T*)dQ, (T*)dtQ, pq, s.q, s.BH * s.M};
    const RmsBwdSide<T> k{(const T*)K, (const T*)tK, gK, (const T*)dKn, (const T*)dtKn, (T*)dK, (T*)dtK, pk, s.k, s.BH * s.N};
    qk_rmsnorm_jvp_bwd_kernel<T><<<dim3(RMS_BWD_BLOCKS, 2), RMS_THREADS, 0, st>>>(q, k, s.H, s.d, cpr, gs, eps);
    qk_rmsnorm_dg_reduce_kernel<<<2, 1024, 0, st>>>(pq, pk, dgQ, dgK, RMS_BWD_BLOCKS, s.d);
    g_launches += 2;
    return cuda_status(cudaGetLastError());
}

static bool rms_eps_ok(float eps) { return eps >= 0.0f && std::isfinite(eps); }

}  // namespace tvm_attn

using namespace tvm_attn;

extern "C" {

size_t tvm_attn_jvp_workspace_bytes(const tvm_attn_params* p, int is_bwd) {
    Shape s;
    if (check_params(p, &s) != TVM_ATTN_OK) return 0;
    if (!is_bwd) return 0;
    return (size_t)3 * sizeof(float) * (size_t)s.BH * (size_t)s.M;   // per query row
}

int tvm_attn_jvp_fwd(const tvm_attn_params* p, const void* Q, const void* K, const void* V, const void* tQ,
                     const void* tK, const void* tV, void* O, void* tO, float* lse, float* mu, void* workspace,
                     size_t workspace_bytes, void* cuda_stream) {
    (void)workspace; (void)workspace_bytes;
    Shape s;
    int rc = check_params(p, &s);
    if (rc != TVM_ATTN_OK) return rc;
    const void* ptrs[] = {Q, K, V, tQ, tK, tV, O, tO, lse, mu};
    for (const void* x : ptrs)
        if (!x || !aligned16(x)) return TVM_ATTN_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    g_prof.begin_call();
    if (s.simt) {
        return s.fp32 ? simt_fwd<float>(s, Q, K, V, tQ, tK, tV, O, tO, lse, mu, st)
                      : simt_fwd<__nv_bfloat16>(s, Q, K, V, tQ, tK, tV, O, tO, lse, mu, st);
    }
    rc = device_is_sm100();
    if (rc != TVM_ATTN_OK) return rc;
    int* status = status_word_ptr();
    if (!status) return TVM_ATTN_CUDA_ERROR;
    const void* strm[4] = {K, tK, V, tV};
    if (s.dp <= 80) {
        FwdParams f;
        f.d = s.d; f.BH = (int)s.BH; f.H = s.H; f.q = s.q; f.k = s.k;
        f.alpha = s.alpha; f.c2 = s.alpha * 1.4426950408889634f;
        f.Q = static_cast<const __nv_bfloat16*>(Q); f.tQ = static_cast<const __nv_bfloat16*>(tQ);
        f.K = static_cast<const __nv_bfloat16*>(K); f.tK = static_cast<const __nv_bfloat16*>(tK);
        f.V = static_cast<const __nv_bfloat16*>(V); f.tV = static_cast<const __nv_bfloat16*>(tV);
        f.O = static_cast<__nv_bfloat16*>(O); f.tO = static_cast<__nv_bfloat16*>(tO);
        f.lse = lse; f.mu = mu; f.status = status;
        switch (s.dp) {
            case 16: return launch_fwd<16>(s, strm, f, st);
            case 32: return launch_fwd<32>(s, strm, f, st);
            case 48: return launch_fwd<48>(s, strm, f, st);
            case 64: return launch_fwd<64>(s, strm, f, st);
            default: return launch_fwd<80>(s, strm, f, st);
        }
    }
    if (!s.plain) return TVM_ATTN_UNSUPPORTED;  // head dims above 80: self-attention on packed tensors only
    TcParams prm = base_params(s, status);
    prm.out0 = O; prm.out1 = tO; prm.lse_out = lse; prm.mu_out = mu;
    const void* own[4] = {Q, tQ, Q, tQ};
    return launch_tc_na<MODE_FWD>(s, own, strm, prm, st);
}

int tvm_attn_jvp_bwd(const tvm_attn_params* p, const void* Q, const void* K, const void* V, const void* tQ,
                     const void* tK, const void* tV, const void* O, const void* tO, const float* lse, const float* mu,
                     const void* dO, const void* dtO, void* dQ, void* dK, void* dV, void* dtQ, void* dtK, void* dtV,
                     void* workspace, size_t workspace_bytes, void* cuda_stream) {
    Shape s;
    int rc = check_params(p, &s);
    if (rc != TVM_ATTN_OK) return rc;
    const void* ptrs[] = {Q, K, V, tQ, tK, tV, O, tO, lse, mu, dQ, dK, dV, workspace};
    for (const void* x : ptrs)
        if (!x || !aligned16(x)) return TVM_ATTN_INVALID_ARG;
    // A null cotangent means zero (dtO null = the "detach JVP" setting: no gradient through tO).  With dtO null the
    // tangent gradients are identically zero and their outputs may be null too.
    if (!dO && !dtO) return TVM_ATTN_INVALID_ARG;
    const void* opt[] = {dO, dtO, dtQ, dtK, dtV};
    for (const void* x : opt)
        if (x && !aligned16(x)) return TVM_ATTN_INVALID_ARG;
    if (dtO && (!dtQ || !dtK || !dtV)) return TVM_ATTN_INVALID_ARG;
    const int absent = (dtO ? 0 : ABSENT_HC) | (dO ? 0 : ABSENT_G);
    if ((absent || !s.plain) && !s.simt && s.dp > 80) return TVM_ATTN_UNSUPPORTED;  // head dims above 80: both cotangents, packed self-attention
    const size_t rows = (size_t)s.BH * (size_t)s.M;   // query rows: what the workspace and the statistics are sized by
    if (workspace_bytes < 3 * sizeof(float) * rows) return TVM_ATTN_WORKSPACE_TOO_SMALL;
    float* sig1 = static_cast<float*>(workspace);
    float* cvec = sig1 + rows;
    float* lse2 = cvec + rows;  // lse * log2(e)
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    g_prof.begin_call();
    if (!dtO) {  // the tangent gradients of a call without dtO are zero: written here, by none of the passes
        void* zero_out[] = {dtQ, dtK, dtV};
        const int esz = s.fp32 ? 4 : 2, cpr = s.d * esz / 16;
        for (int i = 0; i < 3; ++i) {
            if (!zero_out[i]) continue;
            const Geom& g = i == 0 ? s.q : s.k;
            const long long zr = s.BH * g.rows, n = zr * cpr;
            zero_rows_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(static_cast<uint4*>(zero_out[i]), g, s.H, zr, cpr, 16 / esz);
            g_launches += 1;
            if (cudaGetLastError() != cudaSuccess) return TVM_ATTN_CUDA_ERROR;
        }
    }
    if (s.simt) {
        if (s.fp32) {
            rc = launch_rowsums<float>(s, dO, dtO, O, tO, lse, sig1, cvec, lse2, st);
            if (rc != TVM_ATTN_OK) return rc;
            return simt_bwd<float>(s, Q, K, V, tQ, tK, tV, lse, mu, dO, dtO, sig1, cvec, dQ, dK, dV, dtQ, dtK, dtV, st);
        }
        rc = launch_rowsums<__nv_bfloat16>(s, dO, dtO, O, tO, lse, sig1, cvec, lse2, st);
        if (rc != TVM_ATTN_OK) return rc;
        return simt_bwd<__nv_bfloat16>(s, Q, K, V, tQ, tK, tV, lse, mu, dO, dtO, sig1, cvec, dQ, dK, dV, dtQ, dtK, dtV, st);
    }
    rc = device_is_sm100();
    if (rc != TVM_ATTN_OK) return rc;
    int* status = status_word_ptr();
    if (!status) return TVM_ATTN_CUDA_ERROR;
    rc = launch_rowsums<__nv_bfloat16>(s, dO, dtO, O, tO, lse, sig1, cvec, lse2, st);
    if (rc != TVM_ATTN_OK) return rc;
    if (s.dp <= 80) {
        BwdParams b;
        std::memset(&b, 0, sizeof b);
        b.d = s.d; b.BH = (int)s.BH; b.H = s.H;
        b.alpha = s.alpha; b.c2 = s.alpha * 1.4426950408889634f;
        b.lse2 = lse2; b.mu = mu; b.sig1 = sig1; b.cvec = cvec; b.status = status; b.absent = absent;
        {   // dtV = P^T Hc, dV = P^T G + (P*Nn)^T Hc : owner keys (K, tK); stream queries (Q, tQ | Hc, G)
            BwdParams q = b; q.out_scale = 1.0f;
            q.out0 = dtO ? static_cast<__nv_bfloat16*>(dtV) : nullptr; q.out1 = static_cast<__nv_bfloat16*>(dV);
            const void* own[4] = {K, tK, K, tK};
            const void* strm[4] = {Q, tQ, dtO, dO};
            rc = launch_bwd_pass_dp<BWD_DV>(s, own, strm, q, st);
            if (rc != TVM_ATTN_OK) return rc;
        }
        {   // dtK = alpha W^T Q, dK = alpha (dA^T Q + W^T tQ) : owner keys (K, tK, V, tV); stream (Hc, G | Q, tQ)
            BwdParams q = b; q.out_scale = s.alpha;
            q.out0 = dtO ? static_cast<__nv_bfloat16*>(dtK) : nullptr; q.out1 = static_cast<__nv_bfloat16*>(dK);
            const void* own[4] = {K, tK, V, tV};
            const void* strm[4] = {dtO, dO, Q, tQ};
            rc = launch_bwd_pass_dp<BWD_DK>(s, own, strm, q, st);
            if (rc != TVM_ATTN_OK) return rc;
        }
        {   // dtQ = alpha W K, dQ = alpha (dA K + W tK) : owner queries (Q, tQ, Hc, G); stream (V, tV | K, tK)
            BwdParams q = b; q.out_scale = s.alpha;
            q.out0 = dtO ? static_cast<__nv_bfloat16*>(dtQ) : nullptr; q.out1 = static_cast<__nv_bfloat16*>(dQ);
            const void* own[4] = {Q, tQ, dtO, dO};
            const void* strm[4] = {V, tV, K, tK};
            rc = launch_bwd_pass_dp<BWD_DQ>(s, own, strm, q, st);
        }
        return rc;
    }
    TcParams prm = base_params(s, status);
    prm.lse = lse; prm.mu = mu; prm.sig1 = sig1; prm.cvec = cvec;
    {   // dtV = P^T Hc, dV = P^T G + (P*Nn)^T Hc : owner keys (K, tK), stream queries (Q, tQ | Hc, G)
        TcParams q = prm; q.out0 = dtV; q.out1 = dV;
        const void* own[4] = {K, tK, K, tK};
        const void* strm[4] = {Q, tQ, dtO, dO};
        rc = launch_tc_na<MODE_DV>(s, own, strm, q, st);
        if (rc != TVM_ATTN_OK) return rc;
    }
    {   // dtK = alpha W^T Q, dK = alpha (dA^T Q + W^T tQ) : owner keys (K, tK, V, tV), stream (Q, tQ, Hc, G)
        TcParams q = prm; q.out0 = dtK; q.out1 = dK; q.out_scale = s.alpha;
        const void* own[4] = {K, tK, V, tV};
        const void* strm[4] = {Q, tQ, dtO, dO};
        rc = launch_tc_na<MODE_DK>(s, own, strm, q, st);
        if (rc != TVM_ATTN_OK) return rc;
    }
    {   // dtQ = alpha W K, dQ = alpha (dA K + W tK) : owner queries (Q, tQ, Hc, G), stream (K, tK, V, tV)
        TcParams q = prm; q.out0 = dtQ; q.out1 = dQ; q.out_scale = s.alpha;
        const void* own[4] = {Q, tQ, dtO, dO};
        const void* strm[4] = {K, tK, V, tV};
        rc = launch_tc_na<MODE_DQ>(s, own, strm, q, st);
    }
    return rc;
}

int tvm_attn_jvp_bwd_noalloc(const tvm_attn_params* p, const void* Q, const void* K, const void* V, const void* tQ,
                             const void* tK, const void* tV, const void* O, const void* tO, const float* lse,
                             const float* mu, const void* dO, const void* dtO, void* dQ, void* dK, void* dV, void* dtQ,
                             void* dtK, void* dtV, void* cuda_stream) {
    Shape s;
    const int rc = check_params(p, &s);
    if (rc != TVM_ATTN_OK) return rc;
    if (s.BH * (long long)s.M > (long long)TVM_ATTN_NOALLOC_MAX_ROWS) return TVM_ATTN_TOO_LARGE;
    float* scratch = nullptr;
    const int rs = noalloc_scratch_address(&scratch);
    if (rs != TVM_ATTN_OK) return rs;
    return tvm_attn_jvp_bwd(p, Q, K, V, tQ, tK, tV, O, tO, lse, mu, dO, dtO, dQ, dK, dV, dtQ, dtK, dtV, scratch,
                            sizeof(float) * 3 * (size_t)TVM_ATTN_NOALLOC_MAX_ROWS, cuda_stream);
}

int tvm_attn_check_status(void* cuda_stream) {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return TVM_ATTN_CUDA_ERROR;
    int host = 0;
    if (cudaMemcpyFromSymbol(&host, g_status_word, sizeof(int)) != cudaSuccess) return TVM_ATTN_CUDA_ERROR;
    if (host != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_status_word, &zero, sizeof(int)) != cudaSuccess) return TVM_ATTN_CUDA_ERROR;
        return TVM_ATTN_DEVICE_TIMEOUT;
    }
    return TVM_ATTN_OK;
}

size_t tvm_qk_rmsnorm_jvp_workspace_bytes(const tvm_attn_params* p) {
    Shape s;
    if (check_params(p, &s) != TVM_ATTN_OK) return 0;
    return (size_t)2 * RMS_BWD_BLOCKS * (size_t)s.d * sizeof(float);
}

int tvm_qk_rmsnorm_jvp_fwd(const tvm_attn_params* p, float eps, const void* Q, const void* tQ, const void* K, const void* tK,
                           const float* gQ, const float* gK, void* Qn, void* tQn, void* Kn, void* tKn, void* cuda_stream) {
    Shape s;
    const int rc = check_params(p, &s);
    if (rc != TVM_ATTN_OK) return rc;
    if (!rms_eps_ok(eps)) return TVM_ATTN_INVALID_ARG;
    const void* ptrs[] = {Q, tQ, K, tK, gQ, gK, Qn, tQn, Kn, tKn};
    for (const void* x : ptrs)
        if (!x || !aligned16(x)) return TVM_ATTN_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    return s.fp32 ? rms_fwd<float>(s, eps, Q, tQ, K, tK, gQ, gK, Qn, tQn, Kn, tKn, st)
                  : rms_fwd<__nv_bfloat16>(s, eps, Q, tQ, K, tK, gQ, gK, Qn, tQn, Kn, tKn, st);
}

int tvm_qk_rmsnorm_jvp_bwd(const tvm_attn_params* p, float eps, const void* Q, const void* tQ, const void* K, const void* tK,
                           const float* gQ, const float* gK, const void* dQn, const void* dtQn, const void* dKn,
                           const void* dtKn, void* dQ, void* dtQ, void* dK, void* dtK, float* dgQ, float* dgK, void* workspace,
                           size_t workspace_bytes, void* cuda_stream) {
    Shape s;
    const int rc = check_params(p, &s);
    if (rc != TVM_ATTN_OK) return rc;
    if (!rms_eps_ok(eps)) return TVM_ATTN_INVALID_ARG;
    const void* ptrs[] = {Q, tQ, K, tK, gQ, gK, dQn, dtQn, dKn, dtKn, dQ, dtQ, dK, dtK, dgQ, dgK, workspace};
    for (const void* x : ptrs)
        if (!x || !aligned16(x)) return TVM_ATTN_INVALID_ARG;
    if (workspace_bytes < (size_t)2 * RMS_BWD_BLOCKS * (size_t)s.d * sizeof(float)) return TVM_ATTN_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    float* part = static_cast<float*>(workspace);
    return s.fp32 ? rms_bwd<float>(s, eps, Q, tQ, K, tK, gQ, gK, dQn, dtQn, dKn, dtKn, dQ, dtQ, dK, dtK, dgQ, dgK, part, st)
                  : rms_bwd<__nv_bfloat16>(s, eps, Q, tQ, K, tK, gQ, gK, dQn, dtQn, dKn, dtKn, dQ, dtQ, dK, dtK, dgQ, dgK, part, st);
}

int tvm_attn_selftest_timeout(uint64_t limit_ns, void* cuda_stream) {
    if (limit_ns == 0 || limit_ns > 100ull * 1000ull * 1000ull) return TVM_ATTN_INVALID_ARG;
    int* status = status_word_ptr();
    if (!status) return TVM_ATTN_CUDA_ERROR;
    selftest_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(status, limit_ns);
    g_launches += 1;
    return cuda_status(cudaGetLastError());
}

int tvm_attn_set_profiling(int enable) {
    g_prof.enabled.store(enable != 0);
    g_prof.count.store(0);
    return TVM_ATTN_OK;
}

int tvm_attn_get_profile(float* ms, int capacity) {
    if (!ms || capacity < 0) return TVM_ATTN_INVALID_ARG;
    const int recorded = g_prof.count.load();
    int n = recorded < capacity ? recorded : capacity;
    if (n > 7) n = 7;
    if (n > 0 && cudaEventSynchronize(g_prof.ev[n]) != cudaSuccess) return TVM_ATTN_CUDA_ERROR;
    for (int k = 0; k < n; ++k)
        if (cudaEventElapsedTime(&ms[k], g_prof.ev[k], g_prof.ev[k + 1]) != cudaSuccess) return TVM_ATTN_CUDA_ERROR;
    return n;
}

uint64_t tvm_attn_launch_count(void) { return g_launches.load(); }

const char* tvm_attn_strerror(int code) {
    switch (code) {
        case TVM_ATTN_OK: return "ok";
        case TVM_ATTN_INVALID_ARG: return "invalid argument (null or misaligned pointer, bad dimension, dtype, flags or scale)";
        case TVM_ATTN_UNSUPPORTED: return "unsupported shape or device (need 8 <= d <= 128, d % 8 == 0, an sm_100 GPU)";
        case TVM_ATTN_WORKSPACE_TOO_SMALL: return "workspace smaller than tvm_attn_jvp_workspace_bytes()";
        case TVM_ATTN_CUDA_ERROR: return "a CUDA call or kernel launch failed";
        case TVM_ATTN_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out; outputs are unspecified";
        case TVM_ATTN_TOO_LARGE: return "B*H*N exceeds TVM_ATTN_NOALLOC_MAX_ROWS, the built-in scratch of tvm_attn_jvp_bwd_noalloc; "
                                        "call tvm_attn_jvp_bwd with a workspace instead";
        default: return "unknown status";
    }
}

int tvm_attn_version(void) { return 100; }

}  // extern "C"
