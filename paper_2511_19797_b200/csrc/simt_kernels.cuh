// CUDA-core (FFMA) kernels for the attention-JVP forward and backward.
//
// These are the fp32 validation mode of the library (and, on request, a tensor-core-free way to
// run bf16 tensors).  They use the same algebra and the same saved statistics as the tensor-core
// kernels: an online softmax in the forward (App. C, "Caching softmax statistics") and a
// recompute-per-tile backward split into a row-parallel part (dQ, dtQ) and a column-parallel part
// (dK, dtK, dV, dtV), as App. C "Multi-step backward pass" orders it.
//
// Shape of every kernel: a block owns SIMT_ROWS "owner" rows of one head (queries for the forward
// and the dQ kernel, keys for the dK/dV kernel) and streams the other side through shared memory
// in tiles of 32 rows.  A warp owns SIMT_ROWS/4 owner rows; inside a tile lane j holds the score
// of (owner row, tile row j); output columns c = lane + 32k are accumulated per lane.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>

#include "geometry.cuh"

namespace tvm_attn {

constexpr int SIMT_ROWS = 16;
constexpr int SIMT_TILE = 32;
constexpr int SIMT_THREADS = 128;
constexpr int SIMT_RPW = SIMT_ROWS / (SIMT_THREADS / 32);  // owner rows per warp
constexpr int SIMT_MAXK = 4;                               // ceil(128 / 32) output columns per lane

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f32(float* p, float v) { *p = v; }
__device__ __forceinline__ void from_f32(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// Copies `rows` rows of a head (N rows of d elements, `rs` elements apart) starting at row r0 into shared memory
// with row pitch `pitch` floats; rows at or beyond N are filled with zeros.
// A null `tensor` (an absent cotangent) reads as zeros.
template <typename T>
__device__ __forceinline__ void load_rows(float* dst, const T* tensor, size_t head_off, long long rs, int r0, int rows, int N, int d, int pitch) {
    for (int idx = threadIdx.x; idx < rows * d; idx += SIMT_THREADS) {
        const int r = idx / d, c = idx - r * d;
        const int gr = r0 + r;
        dst[r * pitch + c] = (tensor && gr < N) ? to_f32(tensor[head_off + (size_t)gr * rs + c]) : 0.0f;
    }
}

// ------------------------------------------------------------------------------------------------
// Forward: O, tO, lse, mu.
template <typename T>
__global__ void __launch_bounds__(SIMT_THREADS)
simt_fwd_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
                const T* __restrict__ tQ, const T* __restrict__ tK, const T* __restrict__ tV,
                T* __restrict__ O, T* __restrict__ tO, float* __restrict__ lse, float* __restrict__ mu,
                Geom qg, Geom kg, int H, int d, float alpha) {
    extern __shared__ float smem[];
    const int pitch = d + 1;
    float* sq = smem;                       // [SIMT_ROWS][d]
    float* stq = sq + SIMT_ROWS * d;        // [SIMT_ROWS][d]
    float* sk = stq + SIMT_ROWS * d;        // [SIMT_TILE][pitch] each
    float* stk = sk + SIMT_TILE * pitch;
    float* sv = stk + SIMT_TILE * pitch;
    float* stv = sv + SIMT_TILE * pitch;

    const int M = qg.rows, N = kg.rows;
    const int tiles = (M + SIMT_ROWS - 1) / SIMT_ROWS;
    const size_t bh = blockIdx.x / tiles;
    const size_t hq = qg.head_off((int)bh, H), hk = kg.head_off((int)bh, H);
    const int i0 = (blockIdx.x % tiles) * SIMT_ROWS;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    load_rows(sq, Q, hq, qg.rs, i0, SIMT_ROWS, M, d, d);
    load_rows(stq, tQ, hq, qg.rs, i0, SIMT_ROWS, M, d, d);

    float m[SIMT_RPW], l[SIMT_RPW], mt[SIMT_RPW];
    float accO[SIMT_RPW][SIMT_MAXK], accR[SIMT_RPW][SIMT_MAXK];
#pragma unroll
    for (int r = 0; r < SIMT_RPW; ++r) {
        m[r] = -CUDART_INF_F; l[r] = 0.f; mt[r] = 0.f;
#pragma unroll
        for (int k = 0; k < SIMT_MAXK; ++k) { accO[r][k] = 0.f; accR[r][k] = 0.f; }
    }

    for (int j0 = 0; j0 < N; j0 += SIMT_TILE) {
        __syncthreads();
        load_rows(sk, K, hk, kg.rs, j0, SIMT_TILE, N, d, pitch);
        load_rows(stk, tK, hk, kg.rs, j0, SIMT_TILE, N, d, pitch);
        load_rows(sv, V, hk, kg.rs, j0, SIMT_TILE, N, d, pitch);
        load_rows(stv, tV, hk, kg.rs, j0, SIMT_TILE, N, d, pitch);
        __syncthreads();
        const bool valid = j0 + lane < N;
#pragma unroll
        for (int r = 0; r < SIMT_RPW; ++r) {
            const float* q = sq + (warp * SIMT_RPW + r) * d;
            const float* tq = stq + (warp * SIMT_RPW + r) * d;
            const float* kk = sk + lane * pitch;
            const float* tkk = stk + lane * pitch;
            float s = 0.f, ts = 0.f;
            for (int c = 0; c < d; ++c) {
                const float qv = q[c], kv = kk[c];
                s = fmaf(qv, kv, s);
                ts = fmaf(tq[c], kv, ts);
                ts = fmaf(qv, tkk[c], ts);
            }
            const float a = valid ? alpha * s : -CUDART_INF_F;
            const float t = alpha * ts;
            const float m_new = fmaxf(m[r], warp_max(a));
            const float corr = expf(m[r] - m_new);
            const float p = valid ? expf(a - m_new) : 0.f;
            const float pt = p * t;
            l[r] = l[r] * corr + warp_sum(p);
            mt[r] = mt[r] * corr + warp_sum(pt);
            m[r] = m_new;
#pragma unroll
            for (int k = 0; k < SIMT_MAXK; ++k) { accO[r][k] *= corr; accR[r][k] *= corr; }
            for (int j = 0; j < SIMT_TILE; ++j) {
                const float pj = __shfl_sync(0xffffffffu, p, j);
                const float ptj = __shfl_sync(0xffffffffu, pt, j);
#pragma unroll
                for (int k = 0; k < SIMT_MAXK; ++k) {
                    const int c = lane + 32 * k;
                    if (c < d) {
                        const float vv = sv[j * pitch + c];
                        accO[r][k] = fmaf(pj, vv, accO[r][k]);
                        accR[r][k] = fmaf(ptj, vv, accR[r][k]);
                        accR[r][k] = fmaf(pj, stv[j * pitch + c], accR[r][k]);
                    }
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < SIMT_RPW; ++r) {
        const int i = i0 + warp * SIMT_RPW + r;
        if (i >= M) continue;
        const float inv = 1.0f / l[r];
        const float mun = mt[r] * inv;
#pragma unroll
        for (int k = 0; k < SIMT_MAXK; ++k) {
            const int c = lane + 32 * k;
            if (c < d) {
                const float o = accO[r][k] * inv;
                from_f32(O + hq + (size_t)i * qg.rs + c, o);
                from_f32(tO + hq + (size_t)i * qg.rs + c, fmaf(-mun, o, accR[r][k] * inv));
            }
        }
        if (lane == 0) {
            lse[bh * M + i] = m[r] + logf(l[r]);
            mu[bh * M + i] = mun;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Backward pre-pass (App. C "Step 1", reduced by the identities Sigma_1 = rowsum(dtO*O),
// Sigma_2 = rowsum(dtO*tO) and the standard-attention row term rowsum(dO*O)):
//   sig1[row] = sum_c Hc*O        cvec[row] = sum_c G*O + Hc*tO        lse2[row] = lse[row] * log2(e)
// Pure streaming work (four tensors read once), so it is laid out for the memory system: every lane
// loads 16 bytes per tensor, a row is shared by the smallest power-of-two group of lanes that covers
// its d * sizeof(T) / 16 chunks, and a warp has the loads of ROWSUM_UNROLL row groups in flight
// before it touches the first.
constexpr int ROWSUM_THREADS = 256;
constexpr int ROWSUM_UNROLL = 2;

__device__ __forceinline__ void dot_chunk(const uint4& a, const uint4& b, float& acc, float) {
    const float* x = reinterpret_cast<const float*>(&a);
    const float* y = reinterpret_cast<const float*>(&b);
#pragma unroll
    for (int i = 0; i < 4; ++i) acc = fmaf(x[i], y[i], acc);
}
__device__ __forceinline__ void dot_chunk(const uint4& a, const uint4& b, float& acc, __nv_bfloat16) {
    const __nv_bfloat162* x = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* y = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 xf = __bfloat1622float2(x[i]), yf = __bfloat1622float2(y[i]);
        acc = fmaf(xf.x, yf.x, acc);
        acc = fmaf(xf.y, yf.y, acc);
    }
}

// `gs` = lanes per row = chunks per row `cpr`; rows per warp = 32 / gs (the lanes left over idle).
template <typename T>
__global__ void __launch_bounds__(ROWSUM_THREADS)
bwd_rowsums_kernel(const T* __restrict__ G, const T* __restrict__ Hc, const T* __restrict__ O,
                   const T* __restrict__ tO, const float* __restrict__ lse, float* __restrict__ sig1,
                   float* __restrict__ cvec, float* __restrict__ lse2, long long rows, Geom qg, int H, int d, int cpr,
                   int gs) {
    constexpr int VEC = 16 / (int)sizeof(T);
    const int lane = threadIdx.x & 31;
    const int rpw = 32 / gs;                  // rows per warp and step
    const int sub = lane / gs, c = lane - sub * gs;
    const long long warp_id = (long long)blockIdx.x * (ROWSUM_THREADS / 32) + (threadIdx.x >> 5);
    const long long row0 = warp_id * (ROWSUM_UNROLL * rpw) + sub;
    uint4 g[ROWSUM_UNROLL], h[ROWSUM_UNROLL], o[ROWSUM_UNROLL], t[ROWSUM_UNROLL];
    bool act[ROWSUM_UNROLL];
#pragma unroll
    for (int u = 0; u < ROWSUM_UNROLL; ++u) {
        const long long row = row0 + (long long)u * rpw;
        act[u] = row < rows && c < cpr && sub < rpw;
        g[u] = h[u] = t[u] = make_uint4(0, 0, 0, 0);  // a null G or Hc (absent cotangent) counts as zeros
        if (act[u]) {
            // the statistics are packed (B, H, M); the tensors have strides (H == 0 marks the packed layout: no division)
            size_t off = (size_t)row * d + (size_t)c * VEC;
            if (H > 0) {
                const unsigned bh = (unsigned)row / (unsigned)qg.rows;   // rows fit 31 bits
                off = qg.head_off((int)bh, H) + (size_t)((unsigned)row - bh * (unsigned)qg.rows) * (size_t)qg.rs + (size_t)c * VEC;
            }
            o[u] = __ldg(reinterpret_cast<const uint4*>(O + off));
            if (G) g[u] = __ldg(reinterpret_cast<const uint4*>(G + off));
            if (Hc) {
                h[u] = __ldg(reinterpret_cast<const uint4*>(Hc + off));
                t[u] = __ldg(reinterpret_cast<const uint4*>(tO + off));
            }
        }
    }
#pragma unroll
    for (int u = 0; u < ROWSUM_UNROLL; ++u) {
        const long long row = row0 + (long long)u * rpw;
        float s1 = 0.f, cc = 0.f;
        if (act[u]) {
            dot_chunk(h[u], o[u], s1, T());
            dot_chunk(g[u], o[u], cc, T());
            dot_chunk(h[u], t[u], cc, T());
        }
        s1 = lane_group_sum(s1, gs, lane);
        cc = lane_group_sum(cc, gs, lane);
        if (c == 0 && sub < rpw && row < rows) { sig1[row] = s1; cvec[row] = cc; lse2[row] = lse[row] * 1.4426950408889634f; }
    }
}

// Writes zeros to every row of a tensor with strides (the gradients that are identically zero when a cotangent is
// absent); 16 bytes per thread.
__global__ void __launch_bounds__(256)
zero_rows_kernel(uint4* __restrict__ t, Geom g, int H, long long rows, int chunks_per_row, int elems_per_chunk) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long row = idx / chunks_per_row;
    if (row >= rows) return;
    const int c = (int)(idx - row * chunks_per_row);
    const unsigned bh = (unsigned)row / (unsigned)g.rows;   // rows fit 31 bits
    const size_t off = g.head_off((int)bh, H) + (size_t)((unsigned)row - bh * (unsigned)g.rows) * (size_t)g.rs + (size_t)c * elems_per_chunk;
    t[off / elems_per_chunk] = make_uint4(0, 0, 0, 0);   // every stride is a multiple of 16 bytes
}

// The four per-pair quantities of the backward from the six dot products of a (query, key) pair.
struct PairTerms { float P, Pd, W, dA; };
__device__ __forceinline__ PairTerms pair_terms(bool valid, float alpha, float s, float ts, float Dv, float X,
                                                float lse_i, float mu_i, float sig1_i, float c_i) {
    PairTerms r;
    r.P = valid ? expf(alpha * s - lse_i) : 0.f;
    const float Nn = alpha * ts - mu_i;
    r.Pd = r.P * Nn;
    r.W = r.P * (Dv - sig1_i);
    r.dA = fmaf(r.P, X - c_i, r.W * Nn);
    return r;
}

// ------------------------------------------------------------------------------------------------
// Backward, row-parallel part: dQ = alpha (dA K + W tK), dtQ = alpha W K  (App. C steps 3 and 5).
template <typename T>
__global__ void __launch_bounds__(SIMT_THREADS)
simt_bwd_dq_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
                   const T* __restrict__ tQ, const T* __restrict__ tK, const T* __restrict__ tV,
                   const T* __restrict__ G, const T* __restrict__ Hc, const float* __restrict__ lse,
                   const float* __restrict__ mu, const float* __restrict__ sig1,
                   const float* __restrict__ cvec, T* __restrict__ dQ, T* __restrict__ dtQ, Geom qg, Geom kg, int H,
                   int d, float alpha) {
    extern __shared__ float smem[];
    const int pitch = d + 1;
    float* sq = smem;
    float* stq = sq + SIMT_ROWS * d;
    float* sg = stq + SIMT_ROWS * d;
    float* sh = sg + SIMT_ROWS * d;
    float* sk = sh + SIMT_ROWS * d;
    float* stk = sk + SIMT_TILE * pitch;
    float* sv = stk + SIMT_TILE * pitch;
    float* stv = sv + SIMT_TILE * pitch;

    const int M = qg.rows, N = kg.rows;
    const int tiles = (M + SIMT_ROWS - 1) / SIMT_ROWS;
    const size_t bh = blockIdx.x / tiles;
    const size_t hq = qg.head_off((int)bh, H), hk = kg.head_off((int)bh, H);
    const size_t srow = bh * M;
    const int i0 = (blockIdx.x % tiles) * SIMT_ROWS;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    load_rows(sq, Q, hq, qg.rs, i0, SIMT_ROWS, M, d, d);
    load_rows(stq, tQ, hq, qg.rs, i0, SIMT_ROWS, M, d, d);
    load_rows(sg, G, hq, qg.rs, i0, SIMT_ROWS, M, d, d);
    load_rows(sh, Hc, hq, qg.rs, i0, SIMT_ROWS, M, d, d);

    float st_lse[SIMT_RPW], st_mu[SIMT_RPW], st_s1[SIMT_RPW], st_c[SIMT_RPW];
    float aQ[SIMT_RPW][SIMT_MAXK], aT[SIMT_RPW][SIMT_MAXK];
#pragma unroll
    for (int r = 0; r < SIMT_RPW; ++r) {
        const int i = min(i0 + warp * SIMT_RPW + r, M - 1);
        st_lse[r] = lse[srow + i]; st_mu[r] = mu[srow + i];
        st_s1[r] = sig1[srow + i]; st_c[r] = cvec[srow + i];
#pragma unroll
        for (int k = 0; k < SIMT_MAXK; ++k) { aQ[r][k] = 0.f; aT[r][k] = 0.f; }
    }
    for (int j0 = 0; j0 < N; j0 += SIMT_TILE) {
        __syncthreads();
        load_rows(sk, K, hk, kg.rs, j0, SIMT_TILE, N, d, pitch);
        load_rows(stk, tK, hk, kg.rs, j0, SIMT_TILE, N, d, pitch);
        load_rows(sv, V, hk, kg.rs, j0, SIMT_TILE, N, d, pitch);
        load_rows(stv, tV, hk, kg.rs, j0, SIMT_TILE, N, d, pitch);
        __syncthreads();
        const bool valid = j0 + lane < N;
#pragma unroll
        for (int r = 0; r < SIMT_RPW; ++r) {
            const int ro = (warp * SIMT_RPW + r) * d;
            const int rt = lane * pitch;
            float s = 0.f, ts = 0.f, Dv = 0.f, X = 0.f;
            for (int c = 0; c < d; ++c) {
                const float qv = sq[ro + c], kv = sk[rt + c], hv = sh[ro + c], vv = sv[rt + c];
                s = fmaf(qv, kv, s);
                ts = fmaf(stq[ro + c], kv, ts);
                ts = fmaf(qv, stk[rt + c], ts);
                Dv = fmaf(hv, vv, Dv);
                X = fmaf(sg[ro + c], vv, X);
                X = fmaf(hv, stv[rt + c], X);
            }
            const PairTerms pt = pair_terms(valid, alpha, s, ts, Dv, X, st_lse[r], st_mu[r], st_s1[r], st_c[r]);
            for (int j = 0; j < SIMT_TILE; ++j) {
                const float da = __shfl_sync(0xffffffffu, pt.dA, j);
                const float w = __shfl_sync(0xffffffffu, pt.W, j);
#pragma unroll
                for (int k = 0; k < SIMT_MAXK; ++k) {
                    const int c = lane + 32 * k;
                    if (c < d) {
                        const float kv = sk[j * pitch + c];
                        aQ[r][k] = fmaf(da, kv, aQ[r][k]);
                        aQ[r][k] = fmaf(w, stk[j * pitch + c], aQ[r][k]);
                        aT[r][k] = fmaf(w, kv, aT[r][k]);
                    }
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < SIMT_RPW; ++r) {
        const int i = i0 + warp * SIMT_RPW + r;
        if (i >= M) continue;
#pragma unroll
        for (int k = 0; k < SIMT_MAXK; ++k) {
            const int c = lane + 32 * k;
            if (c < d) {
                from_f32(dQ + hq + (size_t)i * qg.rs + c, alpha * aQ[r][k]);
                if (dtQ) from_f32(dtQ + hq + (size_t)i * qg.rs + c, alpha * aT[r][k]);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Backward, column-parallel part (App. C steps 2, 4 and 6 plus the primal P^T dO):
//   dV = P^T G + Pd^T Hc, dtV = P^T Hc, dK = alpha (dA^T Q + W^T tQ), dtK = alpha W^T Q.
template <typename T>
__global__ void __launch_bounds__(SIMT_THREADS)
simt_bwd_dkv_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
                    const T* __restrict__ tQ, const T* __restrict__ tK, const T* __restrict__ tV,
                    const T* __restrict__ G, const T* __restrict__ Hc, const float* __restrict__ lse,
                    const float* __restrict__ mu, const float* __restrict__ sig1,
                    const float* __restrict__ cvec, T* __restrict__ dK, T* __restrict__ dV,
                    T* __restrict__ dtK, T* __restrict__ dtV, Geom qg, Geom kg, int H, int d, float alpha) {
    extern __shared__ float smem[];
    const int pitch = d + 1;
    float* sk = smem;
    float* stk = sk + SIMT_ROWS * d;
    float* sv = stk + SIMT_ROWS * d;
    float* stv = sv + SIMT_ROWS * d;
    float* sq = stv + SIMT_ROWS * d;
    float* stq = sq + SIMT_TILE * pitch;
    float* sg = stq + SIMT_TILE * pitch;
    float* sh = sg + SIMT_TILE * pitch;

    const int M = qg.rows, N = kg.rows;
    const int tiles = (N + SIMT_ROWS - 1) / SIMT_ROWS;
    const size_t bh = blockIdx.x / tiles;
    const size_t hq = qg.head_off((int)bh, H), hk = kg.head_off((int)bh, H);
    const size_t srow = bh * M;
    const int j0 = (blockIdx.x % tiles) * SIMT_ROWS;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    load_rows(sk, K, hk, kg.rs, j0, SIMT_ROWS, N, d, d);
    load_rows(stk, tK, hk, kg.rs, j0, SIMT_ROWS, N, d, d);
    load_rows(sv, V, hk, kg.rs, j0, SIMT_ROWS, N, d, d);
    load_rows(stv, tV, hk, kg.rs, j0, SIMT_ROWS, N, d, d);

    float aK[SIMT_RPW][SIMT_MAXK], aTK[SIMT_RPW][SIMT_MAXK], aV[SIMT_RPW][SIMT_MAXK], aTV[SIMT_RPW][SIMT_MAXK];
#pragma unroll
    for (int r = 0; r < SIMT_RPW; ++r)
#pragma unroll
        for (int k = 0; k < SIMT_MAXK; ++k) { aK[r][k] = 0.f; aTK[r][k] = 0.f; aV[r][k] = 0.f; aTV[r][k] = 0.f; }

    for (int i0 = 0; i0 < M; i0 += SIMT_TILE) {
        __syncthreads();
        load_rows(sq, Q, hq, qg.rs, i0, SIMT_TILE, M, d, pitch);
        load_rows(stq, tQ, hq, qg.rs, i0, SIMT_TILE, M, d, pitch);
        load_rows(sg, G, hq, qg.rs, i0, SIMT_TILE, M, d, pitch);
        load_rows(sh, Hc, hq, qg.rs, i0, SIMT_TILE, M, d, pitch);
        __syncthreads();
        const bool valid = i0 + lane < M;
        const int i = min(i0 + lane, M - 1);
        const float lse_i = lse[srow + i], mu_i = mu[srow + i], s1_i = sig1[srow + i], c_i = cvec[srow + i];
#pragma unroll
        for (int r = 0; r < SIMT_RPW; ++r) {
            const int ro = (warp * SIMT_RPW + r) * d;
            const int rt = lane * pitch;
            float s = 0.f, ts = 0.f, Dv = 0.f, X = 0.f;
            for (int c = 0; c < d; ++c) {
                const float qv = sq[rt + c], kv = sk[ro + c], hv = sh[rt + c], vv = sv[ro + c];
                s = fmaf(qv, kv, s);
                ts = fmaf(stq[rt + c], kv, ts);
                ts = fmaf(qv, stk[ro + c], ts);
                Dv = fmaf(hv, vv, Dv);
                X = fmaf(sg[rt + c], vv, X);
                X = fmaf(hv, stv[ro + c], X);
            }
            const PairTerms pt = pair_terms(valid, alpha, s, ts, Dv, X, lse_i, mu_i, s1_i, c_i);
            for (int ii = 0; ii < SIMT_TILE; ++ii) {
                const float p = __shfl_sync(0xffffffffu, pt.P, ii);
                const float pd = __shfl_sync(0xffffffffu, pt.Pd, ii);
                const float da = __shfl_sync(0xffffffffu, pt.dA, ii);
                const float w = __shfl_sync(0xffffffffu, pt.W, ii);
#pragma unroll
                for (int k = 0; k < SIMT_MAXK; ++k) {
                    const int c = lane + 32 * k;
                    if (c < d) {
                        const float qv = sq[ii * pitch + c], hv = sh[ii * pitch + c];
                        aV[r][k] = fmaf(p, sg[ii * pitch + c], aV[r][k]);
                        aV[r][k] = fmaf(pd, hv, aV[r][k]);
                        aTV[r][k] = fmaf(p, hv, aTV[r][k]);
                        aK[r][k] = fmaf(da, qv, aK[r][k]);
                        aK[r][k] = fmaf(w, stq[ii * pitch + c], aK[r][k]);
                        aTK[r][k] = fmaf(w, qv, aTK[r][k]);
                    }
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < SIMT_RPW; ++r) {
        const int j = j0 + warp * SIMT_RPW + r;
        if (j >= N) continue;
#pragma unroll
        for (int k = 0; k < SIMT_MAXK; ++k) {
            const int c = lane + 32 * k;
            if (c < d) {
                const size_t o = hk + (size_t)j * kg.rs + c;
                from_f32(dK + o, alpha * aK[r][k]);
                if (dtK) from_f32(dtK + o, alpha * aTK[r][k]);
                from_f32(dV + o, aV[r][k]);
                if (dtV) from_f32(dtV + o, aTV[r][k]);
            }
        }
    }
}

inline size_t simt_smem_bytes(int d, int owner_tensors) {
    return sizeof(float) * ((size_t)owner_tensors * SIMT_ROWS * d + 4 * (size_t)SIMT_TILE * (d + 1));
}

}  // namespace tvm_attn
