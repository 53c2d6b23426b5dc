// Forward kernel of attention with a Jacobian-vector product on sm_100a (tcgen05 + TMEM + TMA),
// for padded head dims up to 80 (d = 72 runs as 80).
//
// Per head (App. C Eq. "sdpa" and the definitions under "Step 1"):
//     S = Q K^T, Sd = tQ K^T + Q tK^T            (three GEMMs per key tile, fp32 accumulators in TMEM)
//     P~ = 2^(c2 S - m), T = alpha Sd             (element-wise warps; m is a lazily updated row reference)
//     O~ += P~ V,  R += (P~ (T - c)) V + P~ tV    (three GEMMs per key tile)
//     O = O~/l,  tO = R/l - (mu - c) O,  lse = ln2 (m + log2 l),  mu = c + sum(P~ (T - c))/l
//
// A work item is 128 query rows of one head, against which the head's keys stream in tiles of 64.  The
// grid has one CTA per SM (a CTA needs the whole tensor memory of one); the items go round-robin over
// the CTAs.  The shared-memory rings, the score buffers and all barrier phases run on through the items,
// so the loads, the operand staging and the first score MMAs of an item are under way while the
// element-wise warps still normalise and store the item before.  (One CTA per item spent a quarter of
// its life on set-up and epilogue at N = 1024.)
//
// What is where
//   * Q and tQ of the CTA's rows are written once into tensor memory as bf16 operands, so the three
//     score GEMMs read only their B operand (the K / tK tile) from shared memory.  With A taken from
//     shared memory a 128 x 64 x 16 MMA would move 6 KB per 32 tensor-pipe cycles, more than the
//     128 B/clk a shared-memory port delivers.
//   * The score accumulators are double-buffered (2 x (64 + 64) columns); the bf16 operands P~ and
//     P~(T - c) are written back over the columns of the accumulators they came from.
//   * 16 element-wise warps: warp w works on TMEM lane quadrant w % 4 (32 query rows) and on the
//     16-column slice w / 4 of every key tile, which is exactly one k-step of the value GEMMs.
//
// Online softmax without a per-tile dependency: the reference m of a row follows the running row
// maximum lazily.  The four warps that share a row exchange their slice maxima through shared memory;
// only when the tile maximum exceeds m by more than FWD_LAZY_LOG2 (rare after the first tile) do they
// take the slow path together: m moves to the new maximum, the centre c of the tangent weights moves
// to T at the new arg-max key, and the accumulators are rescaled, R += (c_old - c_new) O~ keeping them
// consistent.  Centring T keeps the bf16 rounding of P~ (T - c) small where P~ is large, so that
// tO = R/l - (mu - c) O does not cancel badly on rows with a peaked softmax.
//
// Every wait on an mbarrier is bounded; when one gives up the block records a time-out status and
// all roles leave their loops.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "geometry.cuh"
#include "sm100_ptx.cuh"

namespace tvm_attn {

constexpr int FWD_THREADS = 640;        // 4 control warps + 16 element-wise warps
constexpr int FWD_ROWS = 128;           // query rows per CTA
constexpr int FWD_BC = 64;              // keys per tile
constexpr float FWD_LAZY_LOG2 = 3.0f;   // slack of the row reference, in log2 units
constexpr uint64_t FWD_WAIT_LIMIT_NS = 200ull * 1000ull * 1000ull;

struct FwdParams {
    int d, BH, H;
    Geom q, k;    // query side (M rows per head: Q, tQ, O, tO) and key side (N rows: K, tK, V, tV)
    float alpha;  // softmax scale
    float c2;     // alpha * log2(e)
    const __nv_bfloat16* Q;
    const __nv_bfloat16* tQ;
    const __nv_bfloat16* K;   // the four streamed tensors, for the 16-byte copies of columns >= 64
    const __nv_bfloat16* tK;
    const __nv_bfloat16* V;
    const __nv_bfloat16* tV;
    __nv_bfloat16* O;
    __nv_bfloat16* tO;
    float* lse;
    float* mu;
    int* status;  // device status word; non-zero makes the kernel a no-op
};

template <int DP>
struct FwdCfg {
    static_assert(DP % 16 == 0 && DP >= 16 && DP <= 80, "padded head dim must be 16..80");
    static constexpr int KS = DP / 16;            // k-steps of a score GEMM
    static constexpr int NA = DP > 64 ? 2 : 1;    // 64-column swizzle atoms per row
    static constexpr int ST_BYTES = NA * FWD_BC * 128;
    static constexpr int SE = NA == 1 ? 4 : 3;    // stages of the (K, tK) ring
    static constexpr int SL = NA == 1 ? 4 : 3;    // stages of the (V, tV) ring
    static constexpr int TILE_BYTES = (SE + SL) * 2 * ST_BYTES;
    static constexpr int FULL_COUNT = NA;         // TMA issuer (+ the warp copying columns >= 64)
    // barrier slots
    static constexpr int B_EFULL = 0;
    static constexpr int B_EEMPTY = B_EFULL + SE;
    static constexpr int B_LFULL = B_EEMPTY + SE;
    static constexpr int B_LEMPTY = B_LFULL + SL;
    static constexpr int B_SFULL = B_LEMPTY + SL;    // per score buffer: S written (+0, +1), Sd written (+2, +3)
    static constexpr int B_PREADY = B_SFULL + 4;
    static constexpr int B_OUTDONE = B_PREADY + 2;  // per score buffer: the value MMAs that read it have completed
    static constexpr int B_FINAL = B_OUTDONE + 2;
    static constexpr int B_QREADY = B_FINAL + 1;
    static constexpr int B_XMAX = B_QREADY + 1;   // per quadrant: slice maxima exchanged
    static constexpr int B_XSLOW = B_XMAX + 4;    // per quadrant: slow-path / epilogue exchange
    static constexpr int B_DRAIN = B_XSLOW + 4;   // + issuer: used once, while winding down after a time-out
    static constexpr int NBARS = B_DRAIN + 2;
    static_assert(NBARS <= 48, "barrier table too small");
    static constexpr int XMAX_FLOATS = 2 * 128 * 4;   // [parity][row][slice]
    static constexpr int XSLOW_FLOATS = 2 * 128 * 4 * 2;  // [exchange parity][row][slice][2]
    static constexpr int MISC_BYTES = 48 * 8 + 64 + (XMAX_FLOATS + XSLOW_FLOATS) * 4;
    static constexpr int SMEM_BYTES = TILE_BYTES + MISC_BYTES + 1024 /*alignment slack*/;
    // TMEM columns: accumulators O~ and R, the bf16 operands Q and tQ in the gaps behind them, and
    // two score buffers of (S | Sd).
    static constexpr int COL_ACC0 = 0, COL_Q = DP, COL_ACC1 = 128, COL_TQ = 128 + DP, COL_SCORE = 256;
    static constexpr int SCORE_BUF_COLS = 2 * FWD_BC;
    static_assert(DP + DP / 2 <= 128, "operand does not fit behind its accumulator");
};

// Element-wise warps of the forward: `w` in 0..15, TMEM lane quadrant w & 3, column slice w >> 2.
template <int DP>
__device__ __forceinline__ void fwd_elementwise(const FwdParams& p, uint32_t tmem_base, uint32_t bar0,
                                                volatile int* abort_flag, float* xmax, float* xslow, int w, int lane,
                                                int items, int row_tiles, int T) {
    using C = FwdCfg<DP>;
    constexpr int BC = FWD_BC, KS = C::KS;
    auto bar = [&](int i) -> uint32_t { return bar0 + 8u * static_cast<uint32_t>(i); };
    const int q = w & 3, sl = w >> 2;
    const int row = q * 32 + lane;  // query row inside the CTA tile
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16);

    // ---- Q and tQ rows of an item -> bf16 operands in tensor memory (k-step kk at 8 packed columns).  Called
    // once the warp has seen the last scores of the item before: no MMA reads the old operands any more.
    auto stage_q = [&](int item) {
        const int bh_ = item / row_tiles;
        const int row0_ = (item - bh_ * row_tiles) * FWD_ROWS;
        const bool valid_ = row0_ + row < p.q.rows;
        const size_t qoff_ = p.q.head_off(bh_, p.H) + (size_t)(row0_ + row) * (size_t)p.q.rs;
        // the loads of the next chunk are in flight while this one is stored
        auto load = [&](int ch, uint4& v0, uint4& v1) {
            const bool is_t = ch >= KS;
            const int kk = is_t ? ch - KS : ch;
            const __nv_bfloat16* src = (is_t ? p.tQ : p.Q) + qoff_ + 16 * kk;
            v0 = v1 = make_uint4(0, 0, 0, 0);
            if (ch < 2 * KS && valid_ && 16 * kk < p.d) v0 = __ldg(reinterpret_cast<const uint4*>(src));
            if (ch < 2 * KS && valid_ && 16 * kk + 8 < p.d) v1 = __ldg(reinterpret_cast<const uint4*>(src + 8));
        };
        uint4 v0, v1, n0, n1;
        load(sl, v0, v1);
        for (int ch = sl; ch < 2 * KS; ch += 4) {
            load(ch + 4, n0, n1);
            const bool is_t = ch >= KS;
            const int kk = is_t ? ch - KS : ch;
            const uint32_t r[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
            ptx::tmem_st8(lane_addr + (is_t ? C::COL_TQ : C::COL_Q) + 8 * kk, r);
            v0 = n0;
            v1 = n1;
        }
        ptx::tmem_wait_st();
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar(C::B_QREADY));
    };

    int n_slow = 0;  // exchanges done on B_XSLOW
    bool ok = true;
    const uint64_t c2c2 = ptx::pack2(p.c2, p.c2), aa = ptx::pack2(p.alpha, p.alpha);
    float2* xs2 = reinterpret_cast<float2*>(xslow);
    int g = 0, it = 0;  // tiles and items done by this CTA
    if ((int)blockIdx.x < items) stage_q(blockIdx.x);

    for (int item = blockIdx.x; ok && item < items; item += gridDim.x, ++it) {
        const int bh = item / row_tiles;
        const int row0 = (item - bh * row_tiles) * FWD_ROWS;
        const bool row_valid = row0 + row < p.q.rows;
        const size_t grow = (size_t)bh * p.q.rows + row0 + row;   // the statistics are packed (B, H, M)
        const size_t qoff = p.q.head_off(bh, p.H) + (size_t)(row0 + row) * (size_t)p.q.rs;
        float m_ref = -CUDART_INF_F, cen = 0.f;
        uint64_t l2 = 0ull, mt2 = 0ull;  // two partial sums each of P~ and of P~(T - c) over this warp's slices

        for (int j = 0; j < T; ++j, ++g) {
            const int b = g & 1;
            // S is complete before Sd: the row maxima are found and exchanged while the Sd MMAs still run
            if (!ptx::mbar_wait(bar(C::B_SFULL + b), (g >> 1) & 1, abort_flag, FWD_WAIT_LIMIT_NS)) { ok = false; break; }
            ptx::tc_fence_after_sync();
            const uint32_t sbase = lane_addr + C::COL_SCORE + b * C::SCORE_BUF_COLS;
            uint32_t s[16], ts[16];
            ptx::tmem_ld16(sbase + 16 * sl, s);
            ptx::tmem_wait_ld();
            const int nvalid = p.k.rows - j * BC - 16 * sl;  // columns of this slice that are real keys
            if (nvalid < 16) {
#pragma unroll
                for (int c = 0; c < 16; ++c)
                    if (c >= nvalid) s[c] = __float_as_uint(-CUDART_INF_F);
            }
            // slice maximum, exchanged with the three other warps of this quadrant
            float mx = ptx::max3(__uint_as_float(s[0]), __uint_as_float(s[1]), __uint_as_float(s[2]));
#pragma unroll
            for (int c = 3; c < 15; c += 2) mx = ptx::max3(mx, __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
            mx = fmaxf(mx, __uint_as_float(s[15]));
            float* xm = xmax + (g & 1) * 512;
            xm[row * 4 + sl] = mx;
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(C::B_XMAX + q));
            if (!ptx::mbar_wait(bar(C::B_SFULL + 2 + b), (g >> 1) & 1, abort_flag, FWD_WAIT_LIMIT_NS)) { ok = false; break; }
            ptx::tc_fence_after_sync();
            ptx::tmem_ld16(sbase + BC + 16 * sl, ts);
            if (!ptx::mbar_wait(bar(C::B_XMAX + q), g & 1, abort_flag, FWD_WAIT_LIMIT_NS)) { ok = false; break; }
            const float4 o4 = *reinterpret_cast<const float4*>(xm + row * 4);
            const float mrow = fmaxf(ptx::max3(o4.x, o4.y, o4.z), o4.w) * p.c2;  // tile maximum of the row, log2 units
            ptx::tmem_wait_ld();
            const bool need = mrow > m_ref + FWD_LAZY_LOG2;
            if (__any_sync(0xffffffffu, need)) {
                // ---- slow path, taken by the four warps of the quadrant together
                float la = -CUDART_INF_F, lt = 0.f;
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const bool gt = __uint_as_float(s[c]) > la;
                    la = gt ? __uint_as_float(s[c]) : la;
                    lt = gt ? __uint_as_float(ts[c]) : lt;
                }
                float2* xb = xs2 + (n_slow & 1) * 512;  // consecutive exchanges use different halves
                xb[row * 4 + sl] = make_float2(la, lt);
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar(C::B_XSLOW + q));
                if (!ptx::mbar_wait(bar(C::B_XSLOW + q), n_slow & 1, abort_flag, FWD_WAIT_LIMIT_NS)) { ok = false; break; }
                ++n_slow;
                float ba = -CUDART_INF_F, bt = 0.f;
#pragma unroll
                for (int k = 0; k < 4; ++k) {  // ties go to the lowest slice
                    const float2 v = xb[row * 4 + k];
                    const bool gt = v.x > ba;
                    ba = gt ? v.x : ba;
                    bt = gt ? v.y : bt;
                }
                const float tw = bt * p.alpha;
                const float scale = need ? ptx::ex2(m_ref - mrow) : 1.0f;
                const float fix = need ? cen - tw : 0.f;
                if (need) { m_ref = mrow; cen = tw; }
                {
                    float l0, l1, t0, t1;
                    ptx::unpack2(l2, l0, l1);
                    ptx::unpack2(mt2, t0, t1);
                    t0 = scale * fmaf(fix, l0, t0);
                    t1 = scale * fmaf(fix, l1, t1);
                    l0 *= scale;
                    l1 *= scale;
                    l2 = ptx::pack2(l0, l1);
                    mt2 = ptx::pack2(t0, t1);
                }
                if (j > 0) {
                    // accumulators must be at rest: the value MMAs of tile j-1 have completed
                    if (!ptx::mbar_wait(bar(C::B_OUTDONE + ((g - 1) & 1)), ((g - 1) >> 1) & 1, abort_flag, FWD_WAIT_LIMIT_NS)) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    // eight columns at a time: this rare path must not set the register peak of the loop
                    for (int ch = 2 * sl; ch < 2 * KS; ch += 8) {
#pragma unroll 1
                        for (int h = 0; h < 2; ++h) {
                            uint32_t o[8], r[8];
                            ptx::tmem_ld8(lane_addr + C::COL_ACC0 + 8 * (ch + h), o);
                            ptx::tmem_ld8(lane_addr + C::COL_ACC1 + 8 * (ch + h), r);
                            ptx::tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < 8; ++c) {
                                const float ov = __uint_as_float(o[c]);
                                r[c] = __float_as_uint(scale * fmaf(fix, ov, __uint_as_float(r[c])));
                                o[c] = __float_as_uint(scale * ov);
                            }
                            ptx::tmem_st8(lane_addr + C::COL_ACC0 + 8 * (ch + h), o);
                            ptx::tmem_st8(lane_addr + C::COL_ACC1 + 8 * (ch + h), r);
                        }
                    }
                }
            }
            // ---- P~ = 2^(c2 s - m), P~ (T - c); two elements per instruction where the hardware allows
            const uint64_t nm = ptx::pack2(-m_ref, -m_ref), nc = ptx::pack2(-cen, -cen);
            uint32_t pp[8], ppt[8];
#pragma unroll
            for (int c = 0; c < 16; c += 2) {
                const uint64_t x2 = ptx::fma2(ptx::pack2u(s[c], s[c + 1]), c2c2, nm);
                float x0, x1;
                ptx::unpack2(x2, x0, x1);
                const float p0 = ptx::ex2(x0), p1 = ptx::ex2(x1);
                const uint64_t p2 = ptx::pack2(p0, p1);
                const uint64_t t2 = ptx::fma2(ptx::pack2u(ts[c], ts[c + 1]), aa, nc);
                const uint64_t pt2 = ptx::mul2(p2, t2);
                l2 = ptx::add2(l2, p2);
                mt2 = ptx::add2(mt2, pt2);
                float q0, q1;
                ptx::unpack2(pt2, q0, q1);
                pp[c >> 1] = ptx::pack_bf16(p0, p1);
                ppt[c >> 1] = ptx::pack_bf16(q0, q1);
            }
            // operand of k-step `sl` (16 keys) sits at column 16*sl of the accumulator it replaces
            ptx::tmem_st8(sbase + 16 * sl, pp);
            ptx::tmem_st8(sbase + BC + 16 * sl, ppt);
            ptx::tmem_wait_st();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(C::B_PREADY + b));
        }

        if (!ok) break;
        // The next item's operands, so that its loads and first score MMAs run under this item's epilogue.  Their
        // global loads are issued first and land while the row sums are exchanged (which needs no MMA result).
        const bool has_next = item + (int)gridDim.x < items;
        constexpr int NCH = (2 * KS + 3) / 4;  // chunks of 16 columns per warp, at most
        uint4 nq[NCH][2];
        {
            const int nitem = has_next ? item + (int)gridDim.x : item;
            const int bh_ = nitem / row_tiles;
            const int row0_ = (nitem - bh_ * row_tiles) * FWD_ROWS;
            const bool valid_ = has_next && row0_ + row < p.q.rows;
            const size_t qoff_ = p.q.head_off(bh_, p.H) + (size_t)(row0_ + row) * (size_t)p.q.rs;
#pragma unroll
            for (int i = 0; i < NCH; ++i) {
                const int ch = sl + 4 * i;
                const bool is_t = ch >= KS;
                const int kk = is_t ? ch - KS : ch;
                const __nv_bfloat16* src = (is_t ? p.tQ : p.Q) + qoff_ + 16 * kk;
                nq[i][0] = nq[i][1] = make_uint4(0, 0, 0, 0);
                if (ch < 2 * KS && valid_ && 16 * kk < p.d) nq[i][0] = __ldg(reinterpret_cast<const uint4*>(src));
                if (ch < 2 * KS && valid_ && 16 * kk + 8 < p.d) nq[i][1] = __ldg(reinterpret_cast<const uint4*>(src + 8));
            }
        }
        // ---- epilogue: O = O~/l, mu - c = mt/l, tO = R/l - (mu - c) O, lse = ln2 (m + log2 l)
        float2* xe;
        {
            float l0, l1, t0, t1;
            ptx::unpack2(l2, l0, l1);
            ptx::unpack2(mt2, t0, t1);
            xe = xs2 + (n_slow & 1) * 512;
            xe[row * 4 + sl] = make_float2(l0 + l1, t0 + t1);
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(C::B_XSLOW + q));
            ok = ptx::mbar_wait(bar(C::B_XSLOW + q), n_slow & 1, abort_flag, FWD_WAIT_LIMIT_NS);
            ++n_slow;
        }
        if (has_next) {
#pragma unroll
            for (int i = 0; i < NCH; ++i) {
                const int ch = sl + 4 * i;
                if (ch < 2 * KS) {
                    const bool is_t = ch >= KS;
                    const int kk = is_t ? ch - KS : ch;
                    const uint32_t r[8] = {nq[i][0].x, nq[i][0].y, nq[i][0].z, nq[i][0].w, nq[i][1].x, nq[i][1].y, nq[i][1].z, nq[i][1].w};
                    ptx::tmem_st8(lane_addr + (is_t ? C::COL_TQ : C::COL_Q) + 8 * kk, r);
                }
            }
            ptx::tmem_wait_st();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(C::B_QREADY));
        }
        if (ok) ok = ptx::mbar_wait(bar(C::B_FINAL), it & 1, abort_flag, FWD_WAIT_LIMIT_NS);
        if (ok) ptx::tc_fence_after_sync();
        if (ok) {
            float l = 0.f, mt = 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float2 v = xe[row * 4 + k];
                l += v.x;
                mt += v.y;
            }
            const float inv = 1.0f / l;
            const float mun = mt * inv;
            __nv_bfloat16* o_ptr = p.O + qoff;
            __nv_bfloat16* t_ptr = p.tO + qoff;
            for (int ch = sl; ch < KS; ch += 4) {
                uint32_t o[16], r[16];
                ptx::tmem_ld16(lane_addr + C::COL_ACC0 + 16 * ch, o);
                ptx::tmem_ld16(lane_addr + C::COL_ACC1 + 16 * ch, r);
                ptx::tmem_wait_ld();
                uint32_t po[8], pt[8];
#pragma unroll
                for (int c = 0; c < 16; c += 2) {
                    const float o0 = __uint_as_float(o[c]) * inv, o1 = __uint_as_float(o[c + 1]) * inv;
                    const float r0 = fmaf(-mun, o0, __uint_as_float(r[c]) * inv);
                    const float r1 = fmaf(-mun, o1, __uint_as_float(r[c + 1]) * inv);
                    po[c >> 1] = ptx::pack_bf16(o0, o1);
                    pt[c >> 1] = ptx::pack_bf16(r0, r1);
                }
                if (row_valid) {
                    *reinterpret_cast<uint4*>(o_ptr + 16 * ch) = make_uint4(po[0], po[1], po[2], po[3]);
                    *reinterpret_cast<uint4*>(t_ptr + 16 * ch) = make_uint4(pt[0], pt[1], pt[2], pt[3]);
                    if (16 * ch + 8 < p.d) {
                        *reinterpret_cast<uint4*>(o_ptr + 16 * ch + 8) = make_uint4(po[4], po[5], po[6], po[7]);
                        *reinterpret_cast<uint4*>(t_ptr + 16 * ch + 8) = make_uint4(pt[4], pt[5], pt[6], pt[7]);
                    }
                }
            }
            if (sl == 0 && row_valid) {
                p.lse[grow] = (m_ref + log2f(l)) * 0.6931471805599453f;
                p.mu[grow] = cen + mun;
            }
        }
    }
}

template <int DP>
__global__ void __launch_bounds__(FWD_THREADS, 1)
jvp_fwd_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_tk,
               const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_tv,
               const FwdParams p) {
    using C = FwdCfg<DP>;
    constexpr int BC = FWD_BC, KS = C::KS, NA = C::NA, SE = C::SE, SL = C::SL;
    if (*reinterpret_cast<volatile int*>(p.status) != 0) return;  // an earlier kernel timed out

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t e_base = ptx::smem_u32(smem);
    const uint32_t l_base = e_base + SE * 2 * C::ST_BYTES;
    uint8_t* misc = smem + C::TILE_BYTES;
    const uint32_t bar0 = ptx::smem_u32(misc);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 48 * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 48 * 8 + 16);
    float* xmax = reinterpret_cast<float*>(misc + 48 * 8 + 64);
    float* xslow = xmax + C::XMAX_FLOATS;
    auto bar = [&](int i) -> uint32_t { return bar0 + 8u * static_cast<uint32_t>(i); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Work items (a head and 128 of its query rows) go round-robin over the CTAs of a grid that has one
    // CTA per SM.  The rings, the score buffers and every barrier phase run on through the items (tile
    // counter g), so the loads and the first score MMAs of an item are under way while the element-wise
    // warps still write out the item before.
    const int row_tiles = (p.q.rows + FWD_ROWS - 1) / FWD_ROWS;
    const int items = p.BH * row_tiles;
    const int T = (p.k.rows + BC - 1) / BC;  // key tiles per item

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < SE; ++s) { ptx::mbar_init(bar(C::B_EFULL + s), C::FULL_COUNT); ptx::mbar_init(bar(C::B_EEMPTY + s), 1); }
        for (int s = 0; s < SL; ++s) { ptx::mbar_init(bar(C::B_LFULL + s), C::FULL_COUNT); ptx::mbar_init(bar(C::B_LEMPTY + s), 1); }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(bar(C::B_SFULL + b), 1);
            ptx::mbar_init(bar(C::B_SFULL + 2 + b), 1);
            ptx::mbar_init(bar(C::B_PREADY + b), 16);
        }
        ptx::mbar_init(bar(C::B_OUTDONE), 1);
        ptx::mbar_init(bar(C::B_OUTDONE + 1), 1);
        ptx::mbar_init(bar(C::B_FINAL), 1);
        ptx::mbar_init(bar(C::B_QREADY), 16);
        for (int q = 0; q < 4; ++q) { ptx::mbar_init(bar(C::B_XMAX + q), 4); ptx::mbar_init(bar(C::B_XSLOW + q), 4); }
        ptx::mbar_init(bar(C::B_DRAIN), 1);
        ptx::mbar_init(bar(C::B_DRAIN + 1), 1);
        ptx::fence_mbar_init();
    }
    if (NA == 2) {
        // Second swizzle atom of every stage: the 16-byte chunks behind the copied columns must read as
        // zero (they pad d to a multiple of 16) and are never written again.  Logical chunk k of row r
        // sits at physical chunk k ^ (r & 7).
        if (((p.d - 64) >> 3) < 2) {
            for (int i = threadIdx.x; i < (SE + SL) * 2 * BC; i += FWD_THREADS) {
                const int tile = i / BC, r = i - tile * BC;
                uint8_t* atom2 = smem + tile * C::ST_BYTES + BC * 128;
                *reinterpret_cast<uint4*>(atom2 + r * 128 + ((1 ^ (r & 7)) << 4)) = make_uint4(0, 0, 0, 0);
            }
            ptx::fence_proxy_async_smem();
        }
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(tmem_slot), 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    // shared-memory address of tile `t` (0 = K, 1 = tK in the E ring; 2 = V, 3 = tV in the L ring) of iteration j
    auto tile_addr = [&](int t, int j) -> uint32_t {
        return t < 2 ? e_base + ((j % SE) * 2 + t) * C::ST_BYTES : l_base + ((j % SL) * 2 + (t - 2)) * C::ST_BYTES;
    };

    if (warp == 0 || warp == 2) {
        // ------------------------------------------------------------------ producers: warp 0 feeds the
        // (K, tK) ring, warp 2 the (V, tV) ring.  Lane 0 issues the TMA boxes of columns 0..63; all lanes
        // copy the columns from 64 on, 16 bytes per row and chunk (a 64-column TMA box hanging over the
        // end of a 144-byte row would read the next row's bytes from L2 only to replace them by zeros,
        // which nearly doubled the L2 traffic), and signal them one tile later so that two tiles of copies
        // are in flight.
        // Kept to a few dozen instructions per tile: everything that does not depend on the tile (lane's
        // row, chunk positions, source pointers) is set up before the loops.
        const int ring = warp >> 1;
        const int S = ring == 0 ? SE : SL;
        const int b_full = ring == 0 ? C::B_EFULL : C::B_LFULL, b_empty = ring == 0 ? C::B_EEMPTY : C::B_LEMPTY;
        constexpr uint32_t TB = C::ST_BYTES;
        constexpr int KT = NA == 2 ? (DP - 64) / 8 : 1;  // 16-byte chunks per row behind column 64, at most
        const CUtensorMap* map0 = ring == 0 ? &tm_k : &tm_v;
        const CUtensorMap* map1 = ring == 0 ? &tm_tk : &tm_tv;
        const uint32_t ring_base = ring == 0 ? e_base : l_base;
        const __nv_bfloat16* base0 = ring == 0 ? p.K : p.V;
        const __nv_bfloat16* base1 = ring == 0 ? p.tK : p.tV;
        [[maybe_unused]] const int ntail = NA == 2 ? (p.d - 64) >> 3 : 1;
        [[maybe_unused]] const size_t d32 = 32 * (size_t)p.k.rs;             // 32 rows further down, in elements
        [[maybe_unused]] const size_t tile_elems = (size_t)BC * (size_t)p.k.rs;
        [[maybe_unused]] const uint32_t dst_lane = BC * 128 + lane * 128;
        [[maybe_unused]] const uint32_t sw = lane & 7;
        bool ok = true;
        int s = 0, ph = 0, pend_s = -1;
        for (int item = blockIdx.x; ok && item < items; item += gridDim.x) {
            const int bh = item / row_tiles;
            const int cb = bh / p.H, ch = bh - cb * p.H;   // batch and head: coordinates of the 4-D tensor maps
            [[maybe_unused]] const size_t lane_row = p.k.head_off(bh, p.H) + (size_t)lane * (size_t)p.k.rs + 64;
            [[maybe_unused]] const __nv_bfloat16* src0 = base0 + lane_row;
            [[maybe_unused]] const __nv_bfloat16* src1 = base1 + lane_row;
            for (int j = 0; j < T; ++j) {
                if constexpr (NA == 2) {
                    if (pend_s >= 0 && !ptx::mbar_test_warp(bar(b_empty + s), ph ^ 1)) {
                        ptx::cp_async_wait<0>();
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(bar(b_full + pend_s));
                        pend_s = -1;
                    }
                }
                ok = ptx::mbar_wait_warp(bar(b_empty + s), ph ^ 1, abort_flag, FWD_WAIT_LIMIT_NS);
                if (!ok) break;
                const uint32_t stage = ring_base + s * 2 * TB;
                if (lane == 0) {
                    ptx::mbar_arrive_expect_tx(bar(b_full + s), 2 * BC * 128);
                    ptx::tma_load_4d(stage, map0, bar(b_full + s), 0, j * BC, ch, cb);
                    ptx::tma_load_4d(stage + TB, map1, bar(b_full + s), 0, j * BC, ch, cb);
                }
                if constexpr (NA == 2) {
                    const int rows_left = p.k.rows - j * BC;
#pragma unroll
                    for (int k = 0; k < KT; ++k) {
                        if (k < ntail) {
#pragma unroll
                            for (int rp = 0; rp < BC / 32; ++rp) {
                                const bool v = lane + 32 * rp < rows_left;
                                const uint32_t dst = stage + dst_lane + rp * 32 * 128 + ((k ^ sw) << 4);
                                ptx::cp_async_16(dst, v ? src0 + rp * d32 + 8 * k : base0, v ? 16u : 0u);
                                ptx::cp_async_16(dst + TB, v ? src1 + rp * d32 + 8 * k : base1, v ? 16u : 0u);
                            }
                        }
                    }
                    ptx::cp_async_commit();
                    if (pend_s >= 0) {
                        ptx::cp_async_wait<1>();
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(bar(b_full + pend_s));
                    }
                    pend_s = s;
                    src0 += tile_elems;
                    src1 += tile_elems;
                }
                if (++s == S) { s = 0; ph ^= 1; }
            }
        }
        if (NA == 2) {
            ptx::cp_async_wait<0>();  // nothing of ours stays in flight
            if (pend_s >= 0) {       // (also after a time-out: the drain below waits for these barriers)
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar(b_full + pend_s));
            }
        }
        if (!ok) {
            // Winding down after a time-out: the TMA loads this warp started write into this block's shared memory
            // and must have landed before the block exits.  Stages below s carry the phase of this pass over the
            // ring, the others the one before.
            for (int k = 0; k < S; ++k) {
                const bool cur = k < s;
                ptx::mbar_wait_drain(bar(b_full + k), (cur ? ph : ph ^ 1) & 1, ptx::DRAIN_LIMIT_NS);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ score MMAs (warp 1) and value MMAs
        // (warp 3), on two schedulers: an MMA costs 7 to 14 issue slots of its scheduler, which the element-wise
        // warps of that quadrant also need.  Each whole warp runs its loop in converged control flow; one
        // elected lane issues (see mma_ts_elect).
        constexpr uint32_t idesc_s = ptx::idesc_bf16_f32(128, BC, 0, 0);
        const uint32_t tb = __shfl_sync(0xffffffffu, tmem_base, 0);  // warp-uniform for the compiler
        const uint32_t aq = tb + C::COL_Q, atq = tb + C::COL_TQ;
        bool ok = true;
        int g = 0, it = 0;
        for (int item = blockIdx.x; ok && item < items; item += gridDim.x, ++it) {
            // Q, tQ of this item are in tensor memory (the element-wise warps stage them as soon as they have
            // seen the last scores of the item before)
            ok = ptx::mbar_wait_warp(bar(C::B_QREADY), it & 1, abort_flag, FWD_WAIT_LIMIT_NS);
            for (int j = 0; ok && j < T; ++j, ++g) {
                const int b = g & 1;
                ok = ptx::mbar_wait_warp(bar(C::B_EFULL + g % SE), (g / SE) & 1, abort_flag, FWD_WAIT_LIMIT_NS);
                // the score buffer is free once the value MMAs of tile g-2 have read their operands out of it
                if (ok && g >= 2) ok = ptx::mbar_wait_warp(bar(C::B_OUTDONE + b), ((g - 2) >> 1) & 1, abort_flag, FWD_WAIT_LIMIT_NS);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint64_t kd = ptx::smem_desc_sw128(tile_addr(0, g), 16, 1024);
                const uint64_t tkd = ptx::smem_desc_sw128(tile_addr(1, g), 16, 1024);
                const uint32_t dS = tb + C::COL_SCORE + b * C::SCORE_BUF_COLS, dT = dS + BC;
#pragma unroll
                for (int kk = 0; kk < KS; ++kk) {  // S = Q K^T
                    const uint64_t off = (uint64_t)(((kk >> 2) * BC * 128 + (kk & 3) * 32) >> 4);
                    ptx::mma_ts_elect(dS, aq + 8 * kk, kd + off, idesc_s, kk > 0 ? 1u : 0u);
                }
                ptx::mma_commit_elect(bar(C::B_SFULL + b));
#pragma unroll
                for (int kk = 0; kk < KS; ++kk) {  // Sd = tQ K^T
                    const uint64_t off = (uint64_t)(((kk >> 2) * BC * 128 + (kk & 3) * 32) >> 4);
                    ptx::mma_ts_elect(dT, atq + 8 * kk, kd + off, idesc_s, kk > 0 ? 1u : 0u);
                }
#pragma unroll
                for (int kk = 0; kk < KS; ++kk) {  // Sd += Q tK^T
                    const uint64_t off = (uint64_t)(((kk >> 2) * BC * 128 + (kk & 3) * 32) >> 4);
                    ptx::mma_ts_elect(dT, aq + 8 * kk, tkd + off, idesc_s, 1u);
                }
                ptx::mma_commit_elect(bar(C::B_SFULL + 2 + b));
                ptx::mma_commit_elect(bar(C::B_EEMPTY + g % SE));
            }
        }
    } else if (warp == 3) {
        constexpr uint32_t idesc_o = ptx::idesc_bf16_f32(128, DP, 0, 1);
        const uint32_t tb = __shfl_sync(0xffffffffu, tmem_base, 0);
        const uint32_t acc0 = tb + C::COL_ACC0, acc1 = tb + C::COL_ACC1;
        bool ok = true;
        int g = 0;
        for (int item = blockIdx.x; ok && item < items; item += gridDim.x) {
            // The first tile of an item overwrites the accumulators (accumulate = 0): every element-wise warp
            // reads them out for the item before (its epilogue) before it turns to this tile, whose operands
            // the wait below is for.
            for (int j = 0; ok && j < T; ++j, ++g) {
                const int b = g & 1;
                ok = ptx::mbar_wait_warp(bar(C::B_LFULL + g % SL), (g / SL) & 1, abort_flag, FWD_WAIT_LIMIT_NS);
                if (ok) ok = ptx::mbar_wait_warp(bar(C::B_PREADY + b), (g >> 1) & 1, abort_flag, FWD_WAIT_LIMIT_NS);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t a0 = tb + C::COL_SCORE + b * C::SCORE_BUF_COLS, a1 = a0 + BC;
                // MN-major B: atoms of 64 d-columns are BC*128 bytes apart, 8-row groups 1024 bytes apart
                const uint64_t vd = ptx::smem_desc_sw128(tile_addr(2, g), BC * 128, 1024);
                const uint64_t tvd = ptx::smem_desc_sw128(tile_addr(3, g), BC * 128, 1024);
#pragma unroll
                for (int u = 0; u < BC / 16; ++u) {
                    const uint64_t off = (uint64_t)((u * 16 * 128) >> 4);
                    const uint32_t acc = (j > 0 || u > 0) ? 1u : 0u;
                    ptx::mma_ts_elect(acc0, a0 + 16 * u, vd + off, idesc_o, acc);   // O~ += P~ V
                    ptx::mma_ts_elect(acc1, a1 + 16 * u, vd + off, idesc_o, acc);   // R  += P~(T-c) V
                    ptx::mma_ts_elect(acc1, a0 + 16 * u, tvd + off, idesc_o, 1u);   // R  += P~ tV
                }
                ptx::mma_commit_elect(bar(C::B_LEMPTY + g % SL));
                ptx::mma_commit_elect(bar(C::B_OUTDONE + b));
                if (j == T - 1) ptx::mma_commit_elect(bar(C::B_FINAL));
            }
        }
    } else if (warp >= 4) {
        fwd_elementwise<DP>(p, tmem_base, bar0, abort_flag, xmax, xslow, warp - 4, lane, items, row_tiles, T);
    }

    // ---------------------------------------------------------------------- teardown
    if ((warp == 1 || warp == 3) && *abort_flag) {
        // after a time-out: the MMAs this warp queued must be done before the tensor memory is given back
        ptx::mma_commit_elect(bar(C::B_DRAIN + (warp >> 1)));
        ptx::mbar_wait_drain(bar(C::B_DRAIN + (warp >> 1)), 0, ptx::DRAIN_LIMIT_NS);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, 1);
}

}  // namespace tvm_attn
