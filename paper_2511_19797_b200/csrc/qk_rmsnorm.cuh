// RMSNorm QK-normalisation with a tangent, the step in front of the attention of the paper's transformer
// (Sec. 4 "semi-Lipschitz control": RMSNorm as QK-norm with a learnable scale; App. "Lipschitzness of
// RMSNorm" for the definition and the Jacobian), and its backward pass.  Per row x in R^d:
//     r = sqrt(mean(x^2) + eps),  u = x / r,  y = g u,  ty = g (tx / r - u (u . tx) / (d r))
// One launch normalises Q and K, primal and tangent.  Pure streaming work (each tensor is read or written
// once), laid out like the row-sums pre-pass of the attention backward: every lane moves 16 bytes per
// tensor, and a row is shared by the smallest power-of-two group of lanes that covers its chunks.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "geometry.cuh"

namespace tvm_attn {

constexpr int RMS_THREADS = 256;
constexpr int RMS_BWD_BLOCKS = 592;   // blocks per side of the backward: fixed, so that the partial sums of dg
                                      // have a size (and a summation order) that does not depend on the device

template <typename T> struct RmsVec;
template <> struct RmsVec<float> { static constexpr int N = 4; };
template <> struct RmsVec<__nv_bfloat16> { static constexpr int N = 8; };

template <typename T>
__device__ __forceinline__ void rms_load(const T* p, float (&v)[RmsVec<T>::N]);
template <>
__device__ __forceinline__ void rms_load<float>(const float* p, float (&v)[4]) {
    const float4 q = __ldg(reinterpret_cast<const float4*>(p));
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
template <>
__device__ __forceinline__ void rms_load<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 q = __ldg(reinterpret_cast<const uint4*>(p));
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&q);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(h[i]);
        v[2 * i] = f.x;
        v[2 * i + 1] = f.y;
    }
}
__device__ __forceinline__ void rms_store(float* p, const float (&v)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void rms_store(__nv_bfloat16* p, const float (&v)[8]) {
    uint4 q;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&q);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    *reinterpret_cast<uint4*>(p) = q;
}
template <int N>
__device__ __forceinline__ void rms_load_scale(const float* g, float (&v)[N]) {
#pragma unroll
    for (int i = 0; i < N; i += 4) {
        const float4 q = __ldg(reinterpret_cast<const float4*>(g + i));
        v[i] = q.x; v[i + 1] = q.y; v[i + 2] = q.z; v[i + 3] = q.w;
    }
}

template <typename T>
struct RmsFwdSide {
    const T* x; const T* tx; const float* g; T* y; T* ty;
    Geom geom;        // rows per head and strides of this side (Q: M rows, K: N rows)
    long long rows;   // B * H * rows per head
};

// Forward for both sides (blockIdx.y = 0: Q, 1: K).  `cpr` = 16-byte chunks per row, `gs` = lanes per row.
template <typename T>
__global__ void __launch_bounds__(RMS_THREADS)
qk_rmsnorm_jvp_fwd_kernel(const RmsFwdSide<T> q, const RmsFwdSide<T> k, int H, int d, int cpr, int gs, float eps) {
    constexpr int V = RmsVec<T>::N;
    const RmsFwdSide<T>& a = blockIdx.y == 0 ? q : k;
    const int lane = threadIdx.x & 31, rpw = 32 / gs;
    const int sub = lane / gs, c = lane - sub * gs;
    const long long row = ((long long)blockIdx.x * (RMS_THREADS / 32) + (threadIdx.x >> 5)) * rpw + sub;
    const bool act = row < a.rows && c < cpr && sub < rpw;
    float x[V], t[V], g[V];
#pragma unroll
    for (int i = 0; i < V; ++i) x[i] = t[i] = g[i] = 0.f;
    const unsigned bh = (unsigned)row / (unsigned)a.geom.rows;   // rows fit 31 bits
    const size_t off = a.geom.head_off((int)bh, H) + (size_t)((unsigned)row - bh * (unsigned)a.geom.rows) * (size_t)a.geom.rs + (size_t)c * V;
    if (act) {
        rms_load<T>(a.x + off, x);
        rms_load<T>(a.tx + off, t);
        rms_load_scale<V>(a.g + c * V, g);
    }
    float ss = 0.f, s = 0.f;
#pragma unroll
    for (int i = 0; i < V; ++i) { ss = fmaf(x[i], x[i], ss); s = fmaf(x[i], t[i], s); }
    ss = lane_group_sum(ss, gs, lane);
    s = lane_group_sum(s, gs, lane);
    const float inv = 1.0f / sqrtf(ss / (float)d + eps);
    const float m = s * inv * inv / (float)d;   // (u . tx) / (d r)
    if (act) {
        float y[V], ty[V];
#pragma unroll
        for (int i = 0; i < V; ++i) {
            const float u = x[i] * inv;
            y[i] = g[i] * u;
            ty[i] = g[i] * fmaf(-u, m, t[i] * inv);
        }
        rms_store(a.y + off, y);
        rms_store(a.ty + off, ty);
    }
}

template <typename T>
struct RmsBwdSide {
    const T* x; const T* tx; const float* g; const T* dy; const T* dty; T* dx; T* dtx;
    float* partial;   // [RMS_BWD_BLOCKS][d] partial sums of dg
    Geom geom;
    long long rows;
};

// Backward for both sides.  With a = g dy, b = g dty and the row sums ss = x.x, s = x.tx, ax = a.x, bx = b.x,
// bt = b.tx:
//     dtx = (b - u (b.u)/d) / r
//     dx  = (a - u (a.u)/d) / r - (bt x + s b + bx tx) / (d r^3) + 3 bx s x / (d^2 r^5)
//     dg += dy u + dty (tx / r - u s / (d r^2))
// Each block walks over its rows with a fixed stride, every thread keeping the dg terms of its own columns; the
// block then adds them up in a fixed order and writes one partial row; a second kernel adds the partial rows, again
// in a fixed order, so dg is bit-reproducible.
template <typename T>
__global__ void __launch_bounds__(RMS_THREADS, 3)
qk_rmsnorm_jvp_bwd_kernel(const RmsBwdSide<T> q, const RmsBwdSide<T> k, int H, int d, int cpr, int gs, float eps) {
    constexpr int V = RmsVec<T>::N;
    __shared__ float part[(RMS_THREADS / 32) * 32 * V];   // [warp][row in warp][column]; d * rows-per-warp <= 32 * V
    const RmsBwdSide<T>& a = blockIdx.y == 0 ? q : k;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, rpw = 32 / gs;
    const int sub = lane / gs, c = lane - sub * gs;
    const long long rows_per_block = (long long)(RMS_THREADS / 32) * rpw;
    float g[V], dg[V];
#pragma unroll
    for (int i = 0; i < V; ++i) g[i] = dg[i] = 0.f;
    if (c < cpr && sub < rpw) rms_load_scale<V>(a.g + c * V, g);
    const float fd = (float)d;
    const long long rows = a.rows;
    for (long long base = (long long)blockIdx.x * rows_per_block; base < rows; base += (long long)gridDim.x * rows_per_block) {
        const long long row = base + (long long)warp * rpw + sub;
        const bool act = row < rows && c < cpr && sub < rpw;
        float x[V], t[V], gy[V], gt[V];
#pragma unroll
        for (int i = 0; i < V; ++i) x[i] = t[i] = gy[i] = gt[i] = 0.f;
        const unsigned bh = (unsigned)row / (unsigned)a.geom.rows;   // rows fit 31 bits
        const size_t off = a.geom.head_off((int)bh, H) + (size_t)((unsigned)row - bh * (unsigned)a.geom.rows) * (size_t)a.geom.rs + (size_t)c * V;
        if (act) {
            rms_load<T>(a.x + off, x);
            rms_load<T>(a.tx + off, t);
            rms_load<T>(a.dy + off, gy);
            rms_load<T>(a.dty + off, gt);
        }
        float ss = 0.f, s = 0.f, ax = 0.f, bx = 0.f, bt = 0.f;
#pragma unroll
        for (int i = 0; i < V; ++i) {
            const float ai = g[i] * gy[i], bi = g[i] * gt[i];
            ss = fmaf(x[i], x[i], ss);
            s = fmaf(x[i], t[i], s);
            ax = fmaf(ai, x[i], ax);
            bx = fmaf(bi, x[i], bx);
            bt = fmaf(bi, t[i], bt);
        }
        ss = lane_group_sum(ss, gs, lane);
        s = lane_group_sum(s, gs, lane);
        ax = lane_group_sum(ax, gs, lane);
        bx = lane_group_sum(bx, gs, lane);
        bt = lane_group_sum(bt, gs, lane);
        const float inv = 1.0f / sqrtf(ss / fd + eps);
        const float inv2 = inv * inv, k3 = inv2 * inv / fd;
        const float au_d = ax * inv / fd, bu_d = bx * inv / fd;   // (a.u)/d, (b.u)/d
        const float m = s * inv2 / fd;
        const float kx = 3.0f * k3 * bx * s * inv2 / fd - k3 * bt;  // coefficient of x in the terms that differentiate J
        if (act) {
            float dx[V], dtx[V];
#pragma unroll
            for (int i = 0; i < V; ++i) {
                const float ai = g[i] * gy[i], bi = g[i] * gt[i];
                const float u = x[i] * inv;
                dtx[i] = (bi - u * bu_d) * inv;
                dx[i] = (ai - u * au_d) * inv + kx * x[i] - k3 * (s * bi + bx * t[i]);
                dg[i] += gy[i] * u + gt[i] * fmaf(-u, m, t[i] * inv);
            }
            rms_store(a.dx + off, dx);
            rms_store(a.dtx + off, dtx);
        }
    }
    // ---- dg of the block, in a fixed order
    float* mine = part + (warp * rpw + sub) * d + c * V;
    if (c < cpr && sub < rpw) {
#pragma unroll
        for (int i = 0; i < V; ++i) mine[i] = dg[i];
    }
    __syncthreads();
    for (int j = threadIdx.x; j < d; j += RMS_THREADS) {
        float acc = 0.f;
        for (int r = 0; r < (RMS_THREADS / 32) * rpw; ++r) acc += part[r * d + j];
        a.partial[(size_t)blockIdx.x * d + j] = acc;
    }
}

// dg[side][j] = sum over the blocks' partial rows in a fixed order: eight interleaved partial sums per column
// (thread t adds the rows b = t / 128, t / 128 + 8, ...), then those eight in order.
__global__ void __launch_bounds__(1024)
qk_rmsnorm_dg_reduce_kernel(const float* __restrict__ partial_q, const float* __restrict__ partial_k, float* __restrict__ dg_q,
                            float* __restrict__ dg_k, int nblocks, int d) {
    __shared__ float acc8[8][128];
    const float* part = blockIdx.x == 0 ? partial_q : partial_k;
    float* out = blockIdx.x == 0 ? dg_q : dg_k;
    const int j = threadIdx.x & 127, lane8 = threadIdx.x >> 7;
    float acc = 0.f;
    if (j < d)
        for (int b = lane8; b < nblocks; b += 8) acc += part[(size_t)b * d + j];
    acc8[lane8][j] = acc;
    __syncthreads();
    if (lane8 == 0 && j < d) {
        float total = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) total += acc8[k][j];
        out[j] = total;
    }
}

}  // namespace tvm_attn
