// Backward kernels of attention with a Jacobian-vector product on sm_100a (tcgen05 + TMEM + TMA),
// for padded head dims up to 80 (d = 72 runs as 80).  Three passes share one skeleton (App. C
// "Multi-step backward pass" with the standard attention backward for dO summed in):
//
//   pass  owner rows  stream rows  score accumulators (128 x BC fp32)                   bf16 operands A0, A1   acc0, acc1 (128 x d)
//   DV    keys        queries      S^T = K Q^T, Sd^T = tK Q^T + K tQ^T                    P^T, (P Nn)^T          dtV, dV          (step 6)
//   DK    keys        queries      S^T, Sd^T, D^T = V Hc^T, X^T = tV Hc^T + V G^T        W^T, dA^T              dtK/alpha, dK/alpha   (steps 2, 4)
//   DQ    queries     keys         S, Sd, D = Hc V^T, X = G V^T + Hc tV^T                 W, dA                  dtQ/alpha, dQ/alpha   (steps 3, 5)
//
// with P = 2^(c2 S - lse2), Nn = alpha Sd - mu, W = P (D - Sigma1), dA = P (X - c) + W Nn, and
//   acc0 += A0 B0,  acc1 += A1 B0 + A0 B1      (B0, B1 = Hc, G | Q, tQ | K, tK).
//
// A work item is 128 owner rows of one head, against which the other side streams in tiles of BC = 64
// rows.  The grid has one CTA per SM (a CTA needs the whole tensor memory of one); the items go round-robin
// over the CTAs, and the rings, the score buffers and all barrier phases run on through the items, so the
// loads, the operand staging and the first score MMAs of an item overlap the epilogue of the item before.
//
// What is where
//   * The owner operands of the first score pair (K, tK or Q, tQ) are written once into tensor memory
//     as bf16 A operands: with A in tensor memory a 128 x N x 16 MMA runs at full rate for N >= 32,
//     while with A in shared memory it is bound by the shared-memory port (N = 64: 48 clk instead of 32).
//     The owner operands of the second score pair (V, tV or Hc, G) stay in shared memory: tensor
//     memory has no room for them next to the score accumulators.
//   * Score accumulators: DV has two buffers of (S | Sd), so that the MMAs of one tile run under the
//     element-wise work of the other; DK and DQ have one buffer of (S | Sd | D | X) used in two phases
//     (S, Sd are turned into P, Nn in registers and their columns released while D, X are still being
//     computed).  The bf16 operands A0, A1 are written back over accumulator columns the writing warp
//     has read and are consumed from tensor memory by the output MMAs.
//   * 16 element-wise warps: warp w works on TMEM lane quadrant w % 4 (32 owner rows).  DK, DQ: on the
//     16-column slice w / 4 of every tile.  DV: the warps split by tile parity, eight per tile, two
//     slices each.  Nothing is exchanged between them.
//   * Streamed columns 0..63 arrive by TMA; columns from 64 on are 16-byte asynchronous copies (a
//     64-column box hanging over the end of a 144-byte row would read the next row from L2 for nothing).
//     The L-ring producer also copies the per-query statistics of a tile (transposed passes DV, DK).
//   * MMAs are issued by warp 1 (DK, DQ) or by warps 1 and 3 on alternate tiles, ordered by a turn
//     counter (DV).
//
// Every wait on an mbarrier is bounded; when one gives up the block records a time-out status and
// all roles leave their loops.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>
#include <type_traits>

#include "geometry.cuh"
#include "sm100_ptx.cuh"

namespace tvm_attn {

enum : int { BWD_DV = 0, BWD_DK = 1, BWD_DQ = 2 };

constexpr int BWD_THREADS = 640;  // 2 producer + 2 MMA-issuing warps, 16 element-wise warps
constexpr int BWD_ROWS = 128;     // owner rows per CTA
constexpr uint64_t BWD_WAIT_LIMIT_NS = 200ull * 1000ull * 1000ull;

struct BwdParams {
    int d, BH, H;
    Geom o, s;    // owner side and stream side of this pass (DV, DK: keys own, queries stream; DQ: the other way round).
                  // The per-query statistics are packed (B, H, M): indexed by stream rows in DV and DK, by owner rows in DQ.
    float alpha;      // softmax scale
    float c2;         // alpha * log2(e)
    float out_scale;  // factor applied to acc0 / acc1 in the epilogue
    const __nv_bfloat16* own[4];  // owner tensors X0..X3 (X2, X3 unused by DV)
    const __nv_bfloat16* strm[4]; // streamed tensors: E ring (0, 1), L ring (2, 3)
    __nv_bfloat16* out0;          // acc0 destination: dtV | dtK | dtQ
    __nv_bfloat16* out1;          // acc1 destination: dV | dK | dQ
    const float* lse2;  // lse * log2(e), written by the row-sums pre-pass
    const float* mu;
    const float* sig1;  // rowsum(dtO * O)
    const float* cvec;  // rowsum(dO * O) + rowsum(dtO * tO)
    int* status;        // device status word; non-zero makes the kernel a no-op
    // Absent cotangents (a null dO or dtO means zero; Sec. 5.3 "detach JVP" is dtO absent): bit 0 = Hc (dtO),
    // bit 1 = G (dO).  An absent tensor is never loaded; where an MMA still reads its tile (the N = 128 score
    // MMA of DK) the tile's shared memory is zeroed once, where it is an owner operand (DQ) zeros are staged, and
    // the MMAs whose result would be exactly zero are not issued.  out0 may be null when Hc is absent.
    int absent;
};
enum : int { ABSENT_HC = 1, ABSENT_G = 2 };

template <int MODE, int DP>
struct BwdCfg {
    static_assert(DP % 16 == 0 && DP >= 16 && DP <= 80, "padded head dim must be 16..80");
    static constexpr int NPAIR = MODE == BWD_DV ? 1 : 2;   // score pairs
    static constexpr int BC = 64;                          // stream rows per tile
    static constexpr int CW = BC / 4;                      // columns per element-wise warp
    static constexpr bool TRANSPOSED = MODE != BWD_DQ;     // owner rows are keys
    static constexpr int KS = DP / 16;
    static constexpr int NA = DP > 64 ? 2 : 1;             // 64-column swizzle atoms per row
    // Tiles that are only ever read K-major (the shared-memory owner tensors and the E ring) keep the columns
    // from 64 on in an unswizzled block behind the 64-column swizzle atom: [chunk][row][16 bytes], 32 bytes
    // per row instead of a second 128-byte atom.  The L ring is also read MN-major by the output GEMMs, whose
    // single N = DP operand needs one layout: two 128-byte-swizzled atoms.
    static constexpr int OWN_BYTES = BWD_ROWS * 128 + (NA - 1) * BWD_ROWS * 32;  // one owner tensor in shared memory
    static constexpr int NOWN_SMEM = NPAIR == 2 ? 2 : 0;
    // DK, DQ: which owner pair lives in tensor memory.  The second score pair sits on the critical path of a tile
    // (second pair -> element-wise phase B -> output MMAs -> second pair of the next tile) while the first pair
    // runs under it, so the second pair gets the tensor-memory operands (full MMA rate) and the first pair reads
    // its A operands from shared memory (bound by the shared-memory port, but hidden).
    static constexpr int XT0 = NPAIR == 2 ? 2 : 0;  // p.own[XT0], p.own[XT0 + 1] -> tensor memory
    static constexpr int XS0 = NPAIR == 2 ? 0 : 2;  // p.own[XS0], p.own[XS0 + 1] -> shared memory (two-pair passes)
    static constexpr int EST_BYTES = BC * 128 + (NA - 1) * BC * 32;  // one E-ring tile
    static constexpr int LST_BYTES = NA * BC * 128;                  // one L-ring tile
    // Ring depths.  The E ring of DK / DQ (second-pair operands, released right after that pair) is kept shallow: two
    // stages at head dims above 64 measured 2 to 5 % faster than three (and one or a two-stage L ring far slower);
    // at head dims up to 64, three stages in DK and four in DQ.
    static constexpr int SE = NPAIR == 1 ? 4 : (NA == 1 ? (MODE == BWD_DK ? 3 : 4) : 2);
    static constexpr int SL = NA == 1 ? 4 : 3;
    static constexpr int TILE_BYTES = NOWN_SMEM * OWN_BYTES + SE * 2 * EST_BYTES + SL * 2 * LST_BYTES;
    static constexpr int FULL_COUNT = NA;                  // TMA issuer (+ the warp copying columns >= 64)
    // The L-ring producer also copies the per-query statistics of a tile (transposed passes), into a slot
    // that lives and dies with the tile's L stage.
    static constexpr int LFULL_COUNT = (NA == 2 || TRANSPOSED) ? 2 : 1;
    // which ring holds what: the E ring is released after the score MMAs, the L ring after the output MMAs.
    // DV: E = (Q, tQ) score operands, L = (Hc, G) output operands.
    // DK, DQ: E = second-pair score operands (Hc, G | V, tV), L = first-pair score operands that are also
    // the output operands (Q, tQ | K, tK).
    // barrier slots
    static constexpr int B_EFULL = 0;
    static constexpr int B_EEMPTY = B_EFULL + SE;
    static constexpr int B_LFULL = B_EEMPTY + SE;
    static constexpr int B_LEMPTY = B_LFULL + SL;
    static constexpr int B_SFULL = B_LEMPTY + SL;          // DV: per buffer.  DK/DQ: +0 (S, Sd) written, +1 (D, X) written
    static constexpr int B_PREADY = B_SFULL + 2;           // DV: per buffer.  DK/DQ: +0 operands written, +1 (S, Sd) read
    static constexpr int B_FINAL = B_PREADY + 2;
    // Per-item barriers that the two alternating DV issuers wait on come in pairs, one for even and one for odd
    // items of the CTA: with an odd number of tiles per item (or one) an issuer meets only every other item, and
    // a parity wait on a single barrier would then take the completion of the item before last for its own.
    static constexpr int B_QREADY = B_FINAL + 1;   // + (item & 1): the owner operands of the item are in tensor memory
    static constexpr int B_OWNER = B_QREADY + 2;
    static constexpr int B_ACCFREE = B_OWNER + 1;  // + (item & 1): the element-wise warps have read the item's accumulators
    static constexpr int B_OWNFREE = B_ACCFREE + 2;  // the MMAs that read the shared-memory owner tiles of an item are done
    static constexpr int B_DRAIN = B_OWNFREE + 1;    // + issuer: used once, while winding down after a time-out
    static constexpr int NBARS = B_DRAIN + 2;
    static_assert(NBARS <= 48, "barrier table too small");
    static constexpr int STATS_FLOATS = SL * 4 * 64;
    static constexpr int MISC_BYTES = 48 * 8 + 64 + STATS_FLOATS * 4;
    static constexpr int SMEM_BYTES = TILE_BYTES + MISC_BYTES + 1024 /*alignment slack*/;
    // TMEM columns: accumulators, the bf16 owner operands X0, X1 in the gaps behind them, two score buffers
    static constexpr int COL_ACC0 = 0, COL_X0 = DP, COL_ACC1 = 128, COL_X1 = 128 + DP, COL_SCORE = 256;
    // DV: two buffers of (S | Sd).  DK, DQ: one buffer of (S | Sd | D | X), used in two phases.
    static constexpr int SCORE_BUF_COLS = 2 * NPAIR * BC;
    static constexpr int NBUF = NPAIR == 1 ? 2 : 1;
    static_assert(DP + DP / 2 <= 128, "operand does not fit behind its accumulator");
    static_assert(COL_SCORE + NBUF * SCORE_BUF_COLS <= 512, "TMEM over-subscribed");
};

// Element-wise warps of the backward passes: `w` in 0..15.
// HZ: the cotangent Hc = dtO is absent (the "detach JVP" setting), known at compile time: everything that only
// feeds the tangent path is left out -- Sd, Nn, D, W and their MMAs -- and what remains is the standard attention
// backward: P from S, dA = P (G V^T - rowsum(G O)), dV = P^T G, dK = alpha dA^T Q, dQ = alpha dA K.
template <int MODE, int DP, bool HZ>
__device__ __forceinline__ void bwd_elementwise(const BwdParams& p, uint32_t tmem_base, uint32_t bar0,
                                                volatile int* abort_flag, const float* stats, int w, int lane, int items,
                                                int row_tiles, int T) {
    using C = BwdCfg<MODE, DP>;
    constexpr int BC = C::BC, KS = C::KS, NPAIR = C::NPAIR;
    auto bar = [&](int i) -> uint32_t { return bar0 + 8u * static_cast<uint32_t>(i); };
    const int q = w & 3, slot = w >> 2;
    // DK, DQ: every warp works on every tile, on the 16-column slice `slot` (one k-step of the output GEMMs).
    // DV (two score buffers): the warps split by tile parity, eight per tile, two slices each.  A warp then
    // waits half as often for twice the work, and while the eight of one tile wait for their scores the other
    // eight compute: with all sixteen on one tile the issue ports idled through every hand-off.
    const int par = NPAIR == 1 ? (w >> 3) : 0, jstep = NPAIR == 1 ? 2 : 1;
    const int sl = NPAIR == 1 ? 2 * (slot & 1) : slot;  // first (or only) slice of this warp
    const int row = q * 32 + lane;  // owner row inside the CTA tile
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16);

    // ---- owner rows of X0 and X1 of an item -> bf16 operands in tensor memory (k-step kk at 8 packed
    // columns); all of this warp's loads first, then the stores: one global-memory latency instead of one
    // per chunk.  Called once no MMA reads the operands of the item before any more.
    auto stage_x = [&](int item, int item_index) {
        const int bh_ = item / row_tiles;
        const int row0_ = (item - bh_ * row_tiles) * BWD_ROWS;
        const bool valid_ = row0_ + row < p.o.rows;
        const size_t ooff_ = p.o.head_off(bh_, p.H) + (size_t)(row0_ + row) * (size_t)p.o.rs;
        constexpr int NCH = (2 * KS + 3) / 4;  // chunks of 16 columns per warp, at most
        uint4 v[NCH][2];
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int ch = slot + 4 * i;
            const bool second = ch >= KS;
            const int kk = second ? ch - KS : ch;
            const __nv_bfloat16* own = p.own[C::XT0 + (second ? 1 : 0)];  // null: an absent cotangent, staged as zeros
            const __nv_bfloat16* src = own + ooff_ + 16 * kk;
            v[i][0] = v[i][1] = make_uint4(0, 0, 0, 0);
            if (own && ch < 2 * KS && valid_ && 16 * kk < p.d) v[i][0] = __ldg(reinterpret_cast<const uint4*>(src));
            if (own && ch < 2 * KS && valid_ && 16 * kk + 8 < p.d) v[i][1] = __ldg(reinterpret_cast<const uint4*>(src + 8));
        }
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int ch = slot + 4 * i;
            if (ch < 2 * KS) {
                const bool second = ch >= KS;
                const int kk = second ? ch - KS : ch;
                const uint32_t r[8] = {v[i][0].x, v[i][0].y, v[i][0].z, v[i][0].w, v[i][1].x, v[i][1].y, v[i][1].z, v[i][1].w};
                ptx::tmem_st8(lane_addr + (second ? C::COL_X1 : C::COL_X0) + 8 * kk, r);
            }
        }
        ptx::tmem_wait_st();
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar(C::B_QREADY + (item_index & 1)));
    };

    bool ok = true;
    int it = 0;  // items done by this CTA
    if ((int)blockIdx.x < items) stage_x(blockIdx.x, 0);
    // DQ: the statistics of this thread's row in the next item, loaded before the epilogue's stores go out (behind
    // them the loads would wait in the same queue)
    [[maybe_unused]] float n_lse2 = CUDART_INF_F, n_mu = 0.f, n_s1 = 0.f, n_cv = 0.f;
    [[maybe_unused]] auto load_stats = [&](int item_) {
        const int bh_ = item_ / row_tiles;
        const int row0_ = (item_ - bh_ * row_tiles) * BWD_ROWS;
        n_lse2 = CUDART_INF_F; n_mu = 0.f; n_s1 = 0.f; n_cv = 0.f;
        if (row0_ + row < p.o.rows) {
            const size_t grow_ = (size_t)bh_ * p.o.rows + row0_ + row;
            n_lse2 = p.lse2[grow_];
            n_mu = p.mu[grow_];
            n_s1 = p.sig1[grow_];
            n_cv = p.cvec[grow_];
        }
    };
    if (MODE == BWD_DQ && (int)blockIdx.x < items) load_stats(blockIdx.x);
    for (int item = blockIdx.x; ok && item < items; item += gridDim.x, ++it) {
        const int g0 = it * T;  // tiles this CTA has streamed before this item: rings and barrier phases run on
        const int bh = item / row_tiles;
        const int row0 = (item - bh * row_tiles) * BWD_ROWS;
        const bool row_valid = row0 + row < p.o.rows;
        const size_t grow = (size_t)bh * p.o.rows + row0 + row;   // DQ: this query's slot in the packed statistics
        const size_t ooff = p.o.head_off(bh, p.H) + (size_t)(row0 + row) * (size_t)p.o.rs;
        const float r_lse2 = n_lse2, r_mu = n_mu, r_s1 = n_s1, r_cv = n_cv;  // per-row statistics (DQ)
        for (int j = NPAIR == 1 ? ((par ^ g0) & 1) : 0; j < T; j += jstep) {
            const int g = g0 + j;
            const int b = NPAIR == 1 ? (g & 1) : 0, sph = NPAIR == 1 ? (g >> 1) & 1 : (g & 1);
            // the statistics of the tile's queries arrive with its L stage, which is not released before the
            // output MMAs of this tile, hence not before every warp is through with them.  Every wait of these
            // warps is warp-uniform: the tensor-memory accesses behind it need the whole warp.
            const float* st = stats + (g % C::SL) * 4 * 64 + 16 * sl;
            if (NPAIR == 1) {
                // DV waits here for scores that are usually not there yet: a blocking wait, then the statistics'
                // barrier (long complete), and one vote for both
                bool okl = ptx::mbar_wait(bar(C::B_SFULL + b), sph, abort_flag, BWD_WAIT_LIMIT_NS);
                if (okl) okl = ptx::mbar_wait(bar(C::B_LFULL + g % C::SL), (g / C::SL) & 1, abort_flag, BWD_WAIT_LIMIT_NS);
                if (!__all_sync(0xffffffffu, okl)) { ok = false; break; }
            } else if (C::TRANSPOSED) {
                if (!ptx::mbar_wait2_warp(bar(C::B_SFULL + b), sph, bar(C::B_LFULL + g % C::SL), (g / C::SL) & 1, abort_flag, BWD_WAIT_LIMIT_NS)) { ok = false; break; }
            } else {
                if (!ptx::mbar_wait_warp(bar(C::B_SFULL + b), sph, abort_flag, BWD_WAIT_LIMIT_NS)) { ok = false; break; }
            }
            ptx::tc_fence_after_sync();
            const uint32_t sbase = lane_addr + C::COL_SCORE + b * C::SCORE_BUF_COLS + 16 * sl;
            const int key0 = j * BC + 16 * sl;  // first stream row of this slice
            if (NPAIR == 1) {
              const uint64_t c2c2 = ptx::pack2(p.c2, p.c2), aa = ptx::pack2(p.alpha, p.alpha);
#pragma unroll
              for (int sub = 0; sub < 2; ++sub) {  // this warp's two slices
                const uint32_t sb = sbase + 16 * sub;
                const float* stt = st + 16 * sub;
                uint32_t s1[16], s2[16];
                ptx::tmem_ld16(sb, s1);
                if (!HZ) ptx::tmem_ld16(sb + BC, s2);
                ptx::tmem_wait_ld();
                uint32_t pa0[8], pa1[8];
#pragma unroll
                for (int c4 = 0; c4 < 16; c4 += 4) {
                    const float4 l4 = *reinterpret_cast<const float4*>(stt + c4);
                    const float lv[4] = {l4.x, l4.y, l4.z, l4.w};
                    if (HZ) {  // P only
#pragma unroll
                        for (int e = 0; e < 4; e += 2) {
                            const uint64_t x2 = ptx::fma2(ptx::pack2u(s1[c4 + e], s1[c4 + e + 1]), c2c2, ptx::pack2(-lv[e], -lv[e + 1]));
                            float x0, x1;
                            ptx::unpack2(x2, x0, x1);
                            pa0[(c4 + e) >> 1] = ptx::pack_bf16(ptx::ex2(x0), ptx::ex2(x1));
                        }
                        continue;
                    }
                    const float4 m4 = *reinterpret_cast<const float4*>(stt + 64 + c4);
                    const float mv[4] = {m4.x, m4.y, m4.z, m4.w};
#pragma unroll
                    for (int e = 0; e < 4; e += 2) {  // P = 2^(c2 s - lse2), P Nn with Nn = alpha ts - mu: two columns per instruction
                        const uint64_t x2 = ptx::fma2(ptx::pack2u(s1[c4 + e], s1[c4 + e + 1]), c2c2, ptx::pack2(-lv[e], -lv[e + 1]));
                        float x0, x1;
                        ptx::unpack2(x2, x0, x1);
                        const float p0 = ptx::ex2(x0), p1 = ptx::ex2(x1);
                        const uint64_t n2 = ptx::fma2(ptx::pack2u(s2[c4 + e], s2[c4 + e + 1]), aa, ptx::pack2(-mv[e], -mv[e + 1]));
                        const uint64_t q2 = ptx::mul2(ptx::pack2(p0, p1), n2);
                        float q0, q1;
                        ptx::unpack2(q2, q0, q1);
                        pa0[(c4 + e) >> 1] = ptx::pack_bf16(p0, p1);
                        pa1[(c4 + e) >> 1] = ptx::pack_bf16(q0, q1);
                    }
                }
                // operand of a k-step (16 stream rows) sits at the slice's columns of the accumulator it replaces
                ptx::tmem_st8(sb, pa0);
                if (!HZ) ptx::tmem_st8(sb + BC, pa1);
              }
            } else {
                // ---- phase A: P, Nn, -P Sigma1, -P c from (S, Sd), two columns per register pair; then that half of the
                // buffer may be overwritten.  Phase B, which sits on the critical path between the second score pair and
                // the output MMAs, is left with three packed FMAs per column pair.
                uint64_t P2[8], Nn2[8], nPs2[8], nPc2[8];
                {
                    uint32_t s1[16], s2[16];
                    ptx::tmem_ld16(sbase, s1);
                    if (!HZ) ptx::tmem_ld16(sbase + BC, s2);
                    ptx::tmem_wait_ld();
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(bar(C::B_PREADY + 1));
                    const uint64_t c2c2 = ptx::pack2(p.c2, p.c2), aa = ptx::pack2(p.alpha, p.alpha);
#pragma unroll
                    for (int c4 = 0; c4 < 16; c4 += 4) {
                        float lv[4], mv[4], gv[4], cv[4];
                        if (C::TRANSPOSED) {
                            const float4 l4 = *reinterpret_cast<const float4*>(st + c4);
                            const float4 m4 = *reinterpret_cast<const float4*>(st + 64 + c4);
                            const float4 g4 = *reinterpret_cast<const float4*>(st + 128 + c4);
                            const float4 c44 = *reinterpret_cast<const float4*>(st + 192 + c4);
                            lv[0] = l4.x; lv[1] = l4.y; lv[2] = l4.z; lv[3] = l4.w;
                            mv[0] = m4.x; mv[1] = m4.y; mv[2] = m4.z; mv[3] = m4.w;
                            gv[0] = g4.x; gv[1] = g4.y; gv[2] = g4.z; gv[3] = g4.w;
                            cv[0] = c44.x; cv[1] = c44.y; cv[2] = c44.z; cv[3] = c44.w;
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                lv[e] = (key0 + c4 + e < p.s.rows) ? r_lse2 : CUDART_INF_F;  // keys beyond N: P = 0
                                mv[e] = r_mu; gv[e] = r_s1; cv[e] = r_cv;
                            }
                        }
#pragma unroll
                        for (int e = 0; e < 4; e += 2) {
                            const int k = (c4 + e) >> 1;
                            const uint64_t x2 = ptx::fma2(ptx::pack2u(s1[c4 + e], s1[c4 + e + 1]), c2c2, ptx::pack2(-lv[e], -lv[e + 1]));
                            float x0, x1;
                            ptx::unpack2(x2, x0, x1);
                            P2[k] = ptx::pack2(ptx::ex2(x0), ptx::ex2(x1));
                            if (!HZ) {
                                Nn2[k] = ptx::fma2(ptx::pack2u(s2[c4 + e], s2[c4 + e + 1]), aa, ptx::pack2(-mv[e], -mv[e + 1]));
                                nPs2[k] = ptx::mul2(P2[k], ptx::pack2(-gv[e], -gv[e + 1]));
                            }
                            nPc2[k] = ptx::mul2(P2[k], ptx::pack2(-cv[e], -cv[e + 1]));
                        }
                    }
                }
                // ---- phase B: W = P D - P Sigma1, dA = (P X - P c) + W Nn, written over this slice's D and X columns
                if (!ptx::mbar_wait_warp(bar(C::B_SFULL + 1), g & 1, abort_flag, BWD_WAIT_LIMIT_NS)) { ok = false; break; }
                ptx::tc_fence_after_sync();
                uint32_t s3[16], s4[16];
                if (!HZ) ptx::tmem_ld16(sbase + 2 * BC, s3);
                ptx::tmem_ld16(sbase + 3 * BC, s4);
                ptx::tmem_wait_ld();
                uint32_t pa0[8], pa1[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint64_t t2 = ptx::fma2(P2[k], ptx::pack2u(s4[2 * k], s4[2 * k + 1]), nPc2[k]);
                    float d0, d1;
                    if (HZ) {  // dA = P (X - c): no W
                        ptx::unpack2(t2, d0, d1);
                    } else {
                        const uint64_t w2 = ptx::fma2(P2[k], ptx::pack2u(s3[2 * k], s3[2 * k + 1]), nPs2[k]);
                        const uint64_t d2 = ptx::fma2(w2, Nn2[k], t2);
                        float w0, w1;
                        ptx::unpack2(w2, w0, w1);
                        ptx::unpack2(d2, d0, d1);
                        pa0[k] = ptx::pack_bf16(w0, w1);
                    }
                    pa1[k] = ptx::pack_bf16(d0, d1);
                }
                if (!HZ) ptx::tmem_st8(sbase + 2 * BC, pa0);
                ptx::tmem_st8(sbase + 3 * BC, pa1);
            }
            ptx::tmem_wait_st();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(C::B_PREADY + b));
        }
        if (!ok) break;
        // the next item's operands, so that its loads and first score MMAs run under this item's epilogue
        if (item + (int)gridDim.x < items) {
            if (NPAIR == 1) {
                // DV: this warp has seen only the scores of its own tiles; those of the item's last tile, which
                // may belong to the other eight warps, must be complete too before the operands change
                const int gl = g0 + T - 1;
                if (!ptx::mbar_wait_warp(bar(C::B_SFULL + (gl & 1)), (gl >> 1) & 1, abort_flag, BWD_WAIT_LIMIT_NS)) { ok = false; break; }
            }
            stage_x(item + gridDim.x, it + 1);
            if (MODE == BWD_DQ) load_stats(item + gridDim.x);
        }
        if (ok) ok = ptx::mbar_wait_warp(bar(C::B_FINAL), it & 1, abort_flag, BWD_WAIT_LIMIT_NS);
        if (ok) {
            ptx::tc_fence_after_sync();
            // DK: lane pairs write the two rows of the pair one after the other, each as complete 32-byte sectors
            [[maybe_unused]] const bool ok_even = row0 + (row & ~1) < p.o.rows, ok_odd = row0 + (row | 1) < p.o.rows;
            for (int ch = slot; ch < KS; ch += 4) {
                uint32_t x0[16], x1[16];
                ptx::tmem_ld16(lane_addr + C::COL_ACC0 + 16 * ch, x0);
                ptx::tmem_ld16(lane_addr + C::COL_ACC1 + 16 * ch, x1);
                ptx::tmem_wait_ld();
                uint32_t q0[8], q1[8];
#pragma unroll
                for (int c = 0; c < 16; c += 2) {
                    q0[c >> 1] = ptx::pack_bf16(__uint_as_float(x0[c]) * p.out_scale, __uint_as_float(x0[c + 1]) * p.out_scale);
                    q1[c >> 1] = ptx::pack_bf16(__uint_as_float(x1[c]) * p.out_scale, __uint_as_float(x1[c + 1]) * p.out_scale);
                }
                const bool has_hi = 16 * ch + 8 < p.d;
                __nv_bfloat16* p0 = p.out0 + ooff + 16 * ch;  // out0 is null with Hc absent: acc0 was never written, its gradient is zero
                __nv_bfloat16* p1 = p.out1 + ooff + 16 * ch;
                if constexpr (MODE == BWD_DK) {
                    // (measured: DK 2 to 6 % faster this way, DQ the same, DV 2 % slower)
                    store_row_pairs(p1, p.o.rs, lane, ok_even, ok_odd, has_hi, make_uint4(q1[0], q1[1], q1[2], q1[3]), make_uint4(q1[4], q1[5], q1[6], q1[7]));
                    if (p.out0) store_row_pairs(p0, p.o.rs, lane, ok_even, ok_odd, has_hi, make_uint4(q0[0], q0[1], q0[2], q0[3]), make_uint4(q0[4], q0[5], q0[6], q0[7]));
                } else if (row_valid) {
                    *reinterpret_cast<uint4*>(p1) = make_uint4(q1[0], q1[1], q1[2], q1[3]);
                    if (has_hi) *reinterpret_cast<uint4*>(p1 + 8) = make_uint4(q1[4], q1[5], q1[6], q1[7]);
                    if (p.out0) {
                        *reinterpret_cast<uint4*>(p0) = make_uint4(q0[0], q0[1], q0[2], q0[3]);
                        if (has_hi) *reinterpret_cast<uint4*>(p0 + 8) = make_uint4(q0[4], q0[5], q0[6], q0[7]);
                    }
                }
            }
        // the accumulators may be overwritten by the first output MMAs of the next item
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(C::B_ACCFREE + (it & 1)));
        }
    }
}

template <int MODE, int DP, bool HZ>
__global__ void __launch_bounds__(BWD_THREADS, 1)
jvp_bwd_kernel(const __grid_constant__ CUtensorMap tm_s0, const __grid_constant__ CUtensorMap tm_s1,
               const __grid_constant__ CUtensorMap tm_s2, const __grid_constant__ CUtensorMap tm_s3,
               const __grid_constant__ CUtensorMap tm_o2, const __grid_constant__ CUtensorMap tm_o3,
               const BwdParams p) {
    using C = BwdCfg<MODE, DP>;
    constexpr int BC = C::BC, KS = C::KS, NA = C::NA, SE = C::SE, SL = C::SL, NPAIR = C::NPAIR;
    // the next backward pass in the stream, if launched as a programmatic dependent, may start as SMs free up
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (*reinterpret_cast<volatile int*>(p.status) != 0) {  // an earlier kernel timed out
        if (MODE != BWD_DV && threadIdx.x == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
        return;
    }

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t own_base = ptx::smem_u32(smem);
    const uint32_t e_base = own_base + C::NOWN_SMEM * C::OWN_BYTES;
    const uint32_t l_base = e_base + SE * 2 * C::EST_BYTES;
    uint8_t* misc = smem + C::TILE_BYTES;
    const uint32_t bar0 = ptx::smem_u32(misc);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 48 * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 48 * 8 + 16);
    const uint32_t turn_addr = bar0 + 48 * 8 + 32;  // turn counter of the two MMA issuers
    float* stats = reinterpret_cast<float*>(misc + 48 * 8 + 64);  // [stage][4][64]
    auto bar = [&](int i) -> uint32_t { return bar0 + 8u * static_cast<uint32_t>(i); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Work items (a head and 128 of its owner rows) go round-robin over the CTAs of a grid that has one CTA
    // per SM.  The rings, the score buffers and every barrier phase run on through the items (tile counter
    // g), so the loads, the operand staging and the first score MMAs of an item are under way while the
    // element-wise warps still write out the item before.
    const int row_tiles = (p.o.rows + BWD_ROWS - 1) / BWD_ROWS;
    const int items = p.BH * row_tiles;
    const int T = (p.s.rows + BC - 1) / BC;  // stream tiles per item

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        *reinterpret_cast<volatile uint32_t*>(misc + 48 * 8 + 32) = 0u;
        for (int s = 0; s < SE; ++s) { ptx::mbar_init(bar(C::B_EFULL + s), C::FULL_COUNT); ptx::mbar_init(bar(C::B_EEMPTY + s), 1); }
        for (int s = 0; s < SL; ++s) { ptx::mbar_init(bar(C::B_LFULL + s), C::LFULL_COUNT); ptx::mbar_init(bar(C::B_LEMPTY + s), 1); }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(bar(C::B_SFULL + b), 1);
            ptx::mbar_init(bar(C::B_PREADY + b), NPAIR == 1 ? 8 : 16);  // one arrival per warp working on a tile
        }
        ptx::mbar_init(bar(C::B_FINAL), 1);
        ptx::mbar_init(bar(C::B_QREADY), 16);
        ptx::mbar_init(bar(C::B_QREADY + 1), 16);
        ptx::mbar_init(bar(C::B_OWNER), C::FULL_COUNT);
        ptx::mbar_init(bar(C::B_ACCFREE), 16);
        ptx::mbar_init(bar(C::B_ACCFREE + 1), 16);
        ptx::mbar_init(bar(C::B_OWNFREE), 1);
        ptx::mbar_init(bar(C::B_DRAIN), 1);
        ptx::mbar_init(bar(C::B_DRAIN + 1), 1);
        ptx::fence_mbar_init();
    }
    if (NA == 2) {
        // Second swizzle atom of every tile: the 16-byte chunk behind the copied columns must read as zero
        // (it pads d to a multiple of 16) and is never written again.  Logical chunk k of row r sits at
        // physical chunk k ^ (r & 7).
        if (((p.d - 64) >> 3) < 2) {
            for (int i = threadIdx.x; i < C::NOWN_SMEM * BWD_ROWS; i += BWD_THREADS) {  // owners: second chunk block
                const int t = i / BWD_ROWS, r = i - t * BWD_ROWS;
                *reinterpret_cast<uint4*>(smem + t * C::OWN_BYTES + BWD_ROWS * 128 + BWD_ROWS * 16 + r * 16) = make_uint4(0, 0, 0, 0);
            }
            for (int i = threadIdx.x; i < SE * 2 * BC; i += BWD_THREADS) {  // E ring: second chunk block
                const int t = i / BC, r = i - t * BC;
                // stage t / 2, tensor t & 1: second chunk block of the stage's tail area
                *reinterpret_cast<uint4*>(smem + C::NOWN_SMEM * C::OWN_BYTES + (t >> 1) * 2 * C::EST_BYTES + 2 * BC * 128 + 2 * BC * 16 +
                                          (t & 1) * BC * 16 + r * 16) = make_uint4(0, 0, 0, 0);
            }
            for (int i = threadIdx.x; i < SL * 2 * BC; i += BWD_THREADS) {  // L ring: chunk 1 of the second swizzle atom
                const int t = i / BC, r = i - t * BC;
                uint8_t* atom2 = smem + C::NOWN_SMEM * C::OWN_BYTES + SE * 2 * C::EST_BYTES + (t >> 1) * 2 * C::LST_BYTES + (2 + (t & 1)) * BC * 128;
                *reinterpret_cast<uint4*>(atom2 + r * 128 + ((1 ^ (r & 7)) << 4)) = make_uint4(0, 0, 0, 0);
            }
            ptx::fence_proxy_async_smem();
        }
    }
    if (MODE == BWD_DK && p.absent && !HZ) {
        // DK reads both cotangent tiles of an E stage in one N = 128 MMA: the never-loaded one must read as zero
        const int t = (p.absent & ABSENT_HC) ? 0 : 1;
        for (int i = threadIdx.x; i < SE * BC * 8; i += BWD_THREADS) {  // the 64-column atoms, 16 bytes at a time
            const int st = i / (BC * 8), r = i - st * (BC * 8);
            *reinterpret_cast<uint4*>(smem + C::NOWN_SMEM * C::OWN_BYTES + st * 2 * C::EST_BYTES + t * BC * 128 + r * 16) = make_uint4(0, 0, 0, 0);
        }
        if (NA == 2) {
            for (int i = threadIdx.x; i < SE * 2 * BC; i += BWD_THREADS) {  // both chunk blocks of the tail area
                const int st = i / (2 * BC), k = (i / BC) & 1, r = i % BC;
                *reinterpret_cast<uint4*>(smem + C::NOWN_SMEM * C::OWN_BYTES + st * 2 * C::EST_BYTES + 2 * BC * 128 + k * 2 * BC * 16 +
                                          t * BC * 16 + r * 16) = make_uint4(0, 0, 0, 0);
            }
        }
        ptx::fence_proxy_async_smem();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(tmem_slot), 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    // Shared-memory stage of tile j in the E and the L ring.  A stage holds the tile's two tensors interleaved so
    // that, read K-major, the two form ONE operand of 2 * BC rows (a score MMA with N = 128 then covers both):
    //   E stage: [Y0 atom][Y1 atom][tail chunk 0: Y0 rows, Y1 rows][tail chunk 1: Y0 rows, Y1 rows]   (tail: NA == 2)
    //   L stage: [Y0 atom 0][Y1 atom 0][Y0 atom 1][Y1 atom 1]                                            (atom 1: NA == 2)
    auto e_stage = [&](int j) -> uint32_t { return e_base + (j % SE) * 2 * C::EST_BYTES; };
    auto l_stage = [&](int j) -> uint32_t { return l_base + (j % SL) * 2 * C::LST_BYTES; };

    if (warp == 0 || warp == 2) {
        // ------------------------------------------------------------------ producers: warp 0 feeds the E
        // ring (and loads the shared-memory owner tiles first), warp 2 the L ring.  Lane 0 issues the TMA
        // boxes of columns 0..63; all lanes copy the columns from 64 on, 16 bytes per row and chunk, and
        // signal them one tile later so that two tiles of copies are in flight.
        // The element-wise warps leave these warps one issue slot in ten or so, and a stage is refilled no
        // faster than this loop runs, so it is kept to a few dozen instructions per tile: everything that
        // does not depend on the tile (lane's row, chunk positions, source pointers) is set up before it.
        constexpr int KT = NA == 2 ? (DP - 64) / 8 : 1;  // 16-byte chunks per row behind column 64, at most
        const int ntail = NA == 2 ? (p.d - 64) >> 3 : 1;
        const size_t d32 = 32 * (size_t)p.s.rs, d32o = 32 * (size_t)p.o.rs;  // 32 rows further down, in elements (stream, owner)
        bool owner_pend = false;  // owner-tile copies issued (warp 0) and not signalled yet
        auto produce = [&](auto ring_tag) -> void {
            constexpr int ring = decltype(ring_tag)::value;
            constexpr int S = ring == 0 ? SE : SL;
            constexpr int b_full = ring == 0 ? C::B_EFULL : C::B_LFULL, b_empty = ring == 0 ? C::B_EEMPTY : C::B_LEMPTY;
            constexpr uint32_t TB = ring == 0 ? C::EST_BYTES : C::LST_BYTES;
            constexpr bool STATS = ring == 1 && C::TRANSPOSED;  // this ring carries the per-query statistics
            constexpr bool HAS_CP = NA == 2 || STATS;           // the warp copies something itself
            constexpr int NST = 2 * NPAIR;                      // statistics per query: lse2, mu (, Sigma1, c)
            const CUtensorMap* map0 = ring == 0 ? &tm_s0 : &tm_s2;
            const CUtensorMap* map1 = ring == 0 ? &tm_s1 : &tm_s3;
            const uint32_t ring_base = ring == 0 ? e_base : l_base;
            const __nv_bfloat16* base0 = p.strm[2 * ring];
            const __nv_bfloat16* base1 = p.strm[2 * ring + 1];
            // the ring that streams the cotangents (Hc, G): L in DV, E in DK; an absent one is not loaded
            constexpr bool COT = (MODE == BWD_DV && ring == 1) || (MODE == BWD_DK && ring == 0);
            const bool has0 = !COT || !(p.absent & ABSENT_HC), has1 = !COT || !(p.absent & ABSENT_G);
            const uint32_t tx_bytes = ((has0 ? 1 : 0) + (has1 ? 1 : 0)) * BC * 128;
            [[maybe_unused]] const size_t tile_elems = (size_t)BC * (size_t)p.s.rs;
            // Destination of chunk 0 of row `lane` behind the 64-column atom: the E ring keeps compact
            // 16-byte-per-row blocks (K-major operands only), the L ring a second 128-byte-swizzled atom.
            [[maybe_unused]] const uint32_t dst_lane = 2 * BC * 128 + (ring == 0 ? lane * 16 : lane * 128);
            [[maybe_unused]] const uint32_t sw = lane & 7;  // rows 32 apart share it
            // statistics: 16-byte chunks when the rows of the (B, H, N) arrays are 16-byte aligned, else floats
            const bool st16 = (p.s.rows & 3) == 0;
            [[maybe_unused]] const uint32_t st_base = ptx::smem_u32(stats);
            bool ok = true;
            int s = 0, ph = 0, pend_s = -1;  // pend_s: stage of the tile whose copied columns are not signalled yet
            int it = 0;
            for (int item = blockIdx.x; ok && item < items; item += gridDim.x, ++it) {
                const int bh = item / row_tiles;
                [[maybe_unused]] const int row0 = (item - bh * row_tiles) * BWD_ROWS;
                const int cb = bh / p.H, chd = bh - cb * p.H;   // batch and head: coordinates of the 4-D tensor maps
                // element offset of (row `lane`, column 64) in the stream tensors
                [[maybe_unused]] const size_t lane_row = p.s.head_off(bh, p.H) + (size_t)lane * (size_t)p.s.rs + 64;
                [[maybe_unused]] const __nv_bfloat16* src0 = base0 + lane_row;  // advance by one tile per iteration
                [[maybe_unused]] const __nv_bfloat16* src1 = base1 + lane_row;
                [[maybe_unused]] const size_t srow = (size_t)bh * p.s.rows;
                [[maybe_unused]] const float* st_src0 = (lane < 16 ? p.lse2 : p.mu) + srow + 4 * (lane & 15);
                [[maybe_unused]] const float* st_src1 = NST == 4 ? (lane < 16 ? p.sig1 : p.cvec) + srow + 4 * (lane & 15) : nullptr;
                if constexpr (ring == 0 && NPAIR == 2) {
                    // The shared-memory owner tiles of this item, once the MMAs that read those of the item before
                    // are done.  Their copied columns are signalled with the first tile's: nothing needs them earlier.
                    if (it > 0) {
                        if constexpr (HAS_CP) {
                            // the MMAs waited for below need the last tile of the item before: signal its copies first
                            if (pend_s >= 0) {
                                ptx::cp_async_wait<0>();
                                ptx::fence_proxy_async_smem();
                                __syncwarp();
                                if (lane == 0) ptx::mbar_arrive(bar(b_full + pend_s));
                                pend_s = -1;
                                if (owner_pend) {  // an item of one tile: its owner copies were not signalled yet either
                                    if (lane == 0) ptx::mbar_arrive(bar(C::B_OWNER));
                                    owner_pend = false;
                                }
                            }
                        }
                        ok = ptx::mbar_wait_warp(bar(C::B_OWNFREE), (it - 1) & 1, abort_flag, BWD_WAIT_LIMIT_NS);
                        if (!ok) break;
                    }
                    if (lane == 0) {
                        ptx::mbar_arrive_expect_tx(bar(C::B_OWNER), 2 * BWD_ROWS * 128);
                        ptx::tma_load_4d(own_base, &tm_o2, bar(C::B_OWNER), 0, row0, chd, cb);
                        ptx::tma_load_4d(own_base + C::OWN_BYTES, &tm_o3, bar(C::B_OWNER), 0, row0, chd, cb);
                    }
                    if constexpr (NA == 2) {
                        const size_t lane_row_o = p.o.head_off(bh, p.H) + (size_t)(row0 + lane) * (size_t)p.o.rs + 64;
                        const __nv_bfloat16* o2 = p.own[C::XS0] + lane_row_o;
                        const __nv_bfloat16* o3 = p.own[C::XS0 + 1] + lane_row_o;
                        const int rows_left = p.o.rows - row0;
#pragma unroll
                        for (int k = 0; k < KT; ++k) {
                            if (k < ntail) {
#pragma unroll
                                for (int rp = 0; rp < BWD_ROWS / 32; ++rp) {
                                    const bool v = lane + 32 * rp < rows_left;
                                    const uint32_t dst = own_base + BWD_ROWS * 128 + k * BWD_ROWS * 16 + (lane + 32 * rp) * 16;
                                    ptx::cp_async_16(dst, v ? o2 + rp * d32o + 8 * k : p.own[C::XS0], v ? 16u : 0u);
                                    ptx::cp_async_16(dst + C::OWN_BYTES, v ? o3 + rp * d32o + 8 * k : p.own[C::XS0 + 1], v ? 16u : 0u);
                                }
                            }
                        }
                        ptx::cp_async_commit();
                        owner_pend = true;
                    }
                }
                for (int j = 0; j < T; ++j) {
                    if constexpr (HAS_CP) {
                        // Never block on a free stage while a tile's copies are unsignalled: the consumer may need
                        // that tile before it frees the stage.
                        if (pend_s >= 0 && !ptx::mbar_test_warp(bar(b_empty + s), ph ^ 1)) {
                            ptx::cp_async_wait<0>();
                            ptx::fence_proxy_async_smem();
                            __syncwarp();
                            if (lane == 0) ptx::mbar_arrive(bar(b_full + pend_s));
                            pend_s = -1;
                            if (ring == 0 && owner_pend) {  // cp.async groups complete in order: the owner copies have landed too
                                if (lane == 0) ptx::mbar_arrive(bar(C::B_OWNER));
                                owner_pend = false;
                            }
                        }
                    }
                    ok = ptx::mbar_wait_warp(bar(b_empty + s), ph ^ 1, abort_flag, BWD_WAIT_LIMIT_NS);
                    if (!ok) break;
                    const uint32_t stage = ring_base + s * 2 * TB;
                    if (lane == 0) {
                        ptx::mbar_arrive_expect_tx(bar(b_full + s), tx_bytes);
                        if (has0) ptx::tma_load_4d(stage, map0, bar(b_full + s), 0, j * BC, chd, cb);
                        if (has1) ptx::tma_load_4d(stage + BC * 128, map1, bar(b_full + s), 0, j * BC, chd, cb);
                    }
                    if constexpr (HAS_CP) {
                        [[maybe_unused]] const int rows_left = p.s.rows - j * BC;  // rows of this tile that exist
                        if constexpr (STATS) {
                            // queries beyond N read as zero: their rows of the B operands are zero too
                            const uint32_t slot = st_base + s * (4 * 64 * 4);
                            if (st16) {
                                const bool v = 4 * (lane & 15) < rows_left;
                                const uint32_t dst = slot + (lane >> 4) * 256 + (lane & 15) * 16;
                                ptx::cp_async_16(dst, v ? st_src0 + j * BC : p.lse2, v ? 16u : 0u);
                                if (NST == 4) ptx::cp_async_16(dst + 512, v ? st_src1 + j * BC : p.lse2, v ? 16u : 0u);
                            } else {
                                for (int c = lane; c < NST * 64; c += 32) {
                                    const int stat = c >> 6, r = c & 63;
                                    const float* src = (stat == 0 ? p.lse2 : stat == 1 ? p.mu : stat == 2 ? p.sig1 : p.cvec) + srow + j * BC + r;
                                    const bool v = r < rows_left;
                                    ptx::cp_async_4(slot + c * 4, v ? src : p.lse2, v ? 4u : 0u);
                                }
                            }
                        }
#pragma unroll
                        for (int k = 0; k < (NA == 2 ? KT : 0); ++k) {
                            if (k < ntail) {
#pragma unroll
                                for (int rp = 0; rp < BC / 32; ++rp) {
                                    const bool v = lane + 32 * rp < rows_left;
                                    const uint32_t dst = stage + dst_lane +
                                                         (ring == 0 ? k * 2 * BC * 16 + rp * 32 * 16 : rp * 32 * 128 + ((k ^ sw) << 4));
                                    if (has0) ptx::cp_async_16(dst, v ? src0 + rp * d32 + 8 * k : base0, v ? 16u : 0u);
                                    if (has1) ptx::cp_async_16(dst + (ring == 0 ? BC * 16 : BC * 128), v ? src1 + rp * d32 + 8 * k : base1, v ? 16u : 0u);
                                }
                            }
                        }
                        ptx::cp_async_commit();
                        if (pend_s >= 0) {  // the tile before: its copies have had a whole iteration to land
                            ptx::cp_async_wait<1>();
                            ptx::fence_proxy_async_smem();
                            __syncwarp();
                            if (lane == 0) ptx::mbar_arrive(bar(b_full + pend_s));
                            if (ring == 0 && owner_pend) {
                                if (lane == 0) ptx::mbar_arrive(bar(C::B_OWNER));
                                owner_pend = false;
                            }
                        }
                        pend_s = s;
                        if constexpr (NA == 2) {
                            src0 += tile_elems;
                            src1 += tile_elems;
                        }
                    }
                    if (++s == S) { s = 0; ph ^= 1; }
                }
            }
            if (HAS_CP) {
                ptx::cp_async_wait<0>();  // nothing of ours stays in flight
                if (pend_s >= 0) {      // (also after a time-out: the drain below waits for these barriers)
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(bar(b_full + pend_s));
                    if (ring == 0 && owner_pend && lane == 0) ptx::mbar_arrive(bar(C::B_OWNER));
                }
            }
            if (!ok) {
                // Winding down after a time-out: the TMA loads this warp started write into this block's shared
                // memory and must have landed before the block exits.  The last S fills are the ones that may
                // still be in flight: stages below s carry the phase of this pass over the ring, the others the one before.
                for (int k = 0; k < S; ++k) {
                    const bool cur = k < s;
                    if (!cur && it == 0 && ph == 0) continue;  // never filled
                    ptx::mbar_wait_drain(bar(b_full + k), (cur ? ph : ph ^ 1) & 1, ptx::DRAIN_LIMIT_NS);
                }
                if (ring == 0 && NPAIR == 2 && it > 0) ptx::mbar_wait_drain(bar(C::B_OWNER), (it - 1) & 1, ptx::DRAIN_LIMIT_NS);
            }
        };
        if (warp == 0) produce(std::integral_constant<int, 0>{});
        else produce(std::integral_constant<int, 1>{});
    } else if (warp == 1 || warp == 3) {
        // ------------------------------------------------------------------ MMA issuers, warps 1 and 3: each
        // whole warp runs its loop in converged control flow; one elected lane issues (see mma_ts_elect).
        // An issuing thread is held at the rate of the tensor pipe while its MMAs are queued, and the waits
        // and address arithmetic between two steps cost it several hundred clocks next to the element-wise
        // warps of its scheduler; with one issuer that time is added to every tile.  DV: warp 1 takes the
        // even tiles (score buffer 0), warp 3 the odd ones; a tile's output MMAs and the score MMAs that
        // overwrite their operands come from one thread, so the pipe orders them; the accumulating output
        // MMAs of consecutive tiles are ordered by a turn counter.  DK, DQ: warp 1 alone; their one score
        // buffer already serialises the steps.
        const int wsel = warp >> 1;  // 0: warp 1, 1: warp 3
        constexpr uint32_t idesc_s = ptx::idesc_bf16_f32(128, BC, 0, 0);
        constexpr uint32_t idesc_o = ptx::idesc_bf16_f32(128, DP, 0, 1);
        const uint32_t tb = __shfl_sync(0xffffffffu, tmem_base, 0);  // warp-uniform for the compiler
        const uint32_t ax0 = tb + C::COL_X0, ax1 = tb + C::COL_X1;
        // Score MMAs: with the two tensors of a stage forming one K-major operand of 2 * BC rows,
        //   [S | X0 Y1^T] = X0 [Y0 | Y1]^T is ONE N = 128 MMA per k-step and Sd += X1 Y0^T one N = 64 MMA:
        // ten instructions per score pair instead of fifteen (an MMA costs its issuing warp 40 to 70 clocks
        // next to the element-wise warps whatever its size), and the shared-memory port moves A once for both.
        constexpr uint32_t idesc_s2 = ptx::idesc_bf16_f32(128, 2 * BC, 0, 0);
        constexpr uint32_t HI_SW128 = ptx::desc_hi_sw128(1024), HI_TAIL = ptx::desc_hi_nosw(128);
        // low descriptor halves (start address, leading offset); the high half is HI_SW128, or HI_TAIL for the
        // unswizzled block that holds k-step 4 of tiles that are only read K-major
        auto e_klo = [&](uint32_t stage, int kk) -> uint32_t {   // E stage, K-major, rows of Y0 (then Y1)
            return kk < 4 ? ptx::desc_lo(stage, 16) + 2u * kk : ptx::desc_lo(stage + 2 * BC * 128, 2 * BC * 16);
        };
        auto l_klo = [&](uint32_t stage, int kk) -> uint32_t {   // L stage, K-major, rows of Y0 (then Y1)
            return ptx::desc_lo(stage + (kk >> 2) * 2 * BC * 128, 16) + 2u * (kk & 3);
        };
        auto own_klo = [&](uint32_t tile, int kk) -> uint32_t {  // shared-memory owner tile, K-major
            return kk < 4 ? ptx::desc_lo(tile, 16) + 2u * kk : ptx::desc_lo(tile + BWD_ROWS * 128, BWD_ROWS * 16);
        };
        // L stage read MN-major by the output GEMMs (tensor t, k-step u of 16 stream rows): atoms of 64 d-columns
        // are 2 * BC * 128 bytes apart, 8-row groups 1024 bytes apart
        auto l_nlo = [&](uint32_t stage, int t, int u) -> uint32_t {
            return ptx::desc_lo(stage + t * BC * 128, 2 * BC * 128) + (uint32_t)((u * 16 * 128) >> 4);
        };
        auto desc64 = [](uint32_t lo, uint32_t hi) -> uint64_t { return (static_cast<uint64_t>(hi) << 32) | lo; };
        // tiles this CTA streams over all of its items; tile g belongs to item g / T of this CTA
        const int n_it = (int)blockIdx.x < items ? (items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
        const int G = n_it * T;
        // (it, j): item of this CTA and tile inside it, g = it * T + j (kept by the caller: no division per tile)
        auto issue_scores = [&](int g, int it, int j) -> bool {  // DV only (the two-pair passes have their own loop below)
            const int b = g & 1;
            if (!ptx::mbar_wait_warp(bar(C::B_EFULL + g % SE), (g / SE) & 1, abort_flag, BWD_WAIT_LIMIT_NS)) return false;
            // the first tiles of an item: its owner operands are in tensor memory
            if (j < 2 && !ptx::mbar_wait_warp(bar(C::B_QREADY + (it & 1)), (it >> 1) & 1, abort_flag, BWD_WAIT_LIMIT_NS)) return false;
            ptx::tc_fence_after_sync();
            // Y0, Y1 in the E ring, K-major B
            const uint32_t st = e_stage(g);
            const uint32_t dS = tb + C::COL_SCORE + b * C::SCORE_BUF_COLS, dT = dS + BC;
            // (fifteen N = 64 MMAs: here, with every A operand in tensor memory and two issuers, the N = 128 form
            // of the two-pair passes measured 4 to 6 % slower)
            const uint32_t y1 = st + BC * 128, y1t = st + 2 * BC * 128 + BC * 16;  // rows of Y1: atom, tail block
#pragma unroll
            for (int kk = 0; kk < KS; ++kk)  // S = X0 Y0^T
                ptx::mma_ts_elect(dS, ax0 + 8 * kk, desc64(e_klo(st, kk), kk < 4 ? HI_SW128 : HI_TAIL), idesc_s, kk > 0 ? 1u : 0u);
            if (!HZ) {
#pragma unroll
                for (int kk = 0; kk < KS; ++kk)  // Sd = X1 Y0^T
                    ptx::mma_ts_elect(dT, ax1 + 8 * kk, desc64(e_klo(st, kk), kk < 4 ? HI_SW128 : HI_TAIL), idesc_s, kk > 0 ? 1u : 0u);
#pragma unroll
                for (int kk = 0; kk < KS; ++kk)  // Sd += X0 Y1^T
                    ptx::mma_ts_elect(dT, ax0 + 8 * kk,
                                      kk < 4 ? desc64(ptx::desc_lo(y1, 16) + 2u * kk, HI_SW128) : desc64(ptx::desc_lo(y1t, 2 * BC * 16), HI_TAIL),
                                      idesc_s, 1u);
            }
            ptx::mma_commit_elect(bar(C::B_SFULL + b));
            ptx::mma_commit_elect(bar(C::B_EEMPTY + g % SE));
            return true;
        };
        auto issue_outputs = [&](int g, int it, int j) -> bool {  // DV only
            const int b = g & 1;
            if (!ptx::mbar_wait_warp(bar(C::B_LFULL + g % SL), (g / SL) & 1, abort_flag, BWD_WAIT_LIMIT_NS)) return false;
            if (!ptx::mbar_wait_warp(bar(C::B_PREADY + b), (g >> 1) & 1, abort_flag, BWD_WAIT_LIMIT_NS)) return false;
            // the other issuer has queued its batch of tile g - 1: accumulation order is the tile order
            if (!ptx::turn_wait_warp(turn_addr, (uint32_t)g, abort_flag, BWD_WAIT_LIMIT_NS)) return false;
            // the first tile of an item overwrites the accumulators: all sixteen element-wise warps have read them
            if (j == 0 && it > 0 && !ptx::mbar_wait_warp(bar(C::B_ACCFREE + ((it - 1) & 1)), ((it - 1) >> 1) & 1, abort_flag, BWD_WAIT_LIMIT_NS)) return false;
            ptx::tc_fence_after_sync();
            const uint32_t a0 = tb + C::COL_SCORE + b * C::SCORE_BUF_COLS, a1 = a0 + BC;
            // MN-major B (the L ring): atoms of 64 d-columns are BC*128 bytes apart, 8-row groups 1024 bytes apart
            const uint64_t b0 = desc64(l_nlo(l_stage(g), 0, 0), HI_SW128);
            const uint64_t b1 = desc64(l_nlo(l_stage(g), 1, 0), HI_SW128);
            const uint32_t acc0 = tb + C::COL_ACC0, acc1 = tb + C::COL_ACC1;
            if (!HZ && p.absent == 0) {
                // both cotangents present: the loop as plain as it can be (one uniform branch outside it; a branch per
                // MMA inside the unrolled loop costs the issuing warp more than it looks)
#pragma unroll
                for (int u = 0; u < BC / 16; ++u) {
                    const uint64_t off = (uint64_t)((u * 16 * 128) >> 4);
                    const uint32_t acc = (j > 0 || u > 0) ? 1u : 0u;
                    ptx::mma_ts_elect(acc0, a0 + 16 * u, b0 + off, idesc_o, acc);   // acc0 += A0 B0
                    ptx::mma_ts_elect(acc1, a1 + 16 * u, b0 + off, idesc_o, acc);   // acc1 += A1 B0
                    ptx::mma_ts_elect(acc1, a0 + 16 * u, b1 + off, idesc_o, 1u);    // acc1 += A0 B1
                }
            } else if (HZ || (p.absent & ABSENT_HC)) {  // B0 = Hc absent
#pragma unroll
                for (int u = 0; u < BC / 16; ++u) {
                    const uint64_t off = (uint64_t)((u * 16 * 128) >> 4);
                    ptx::mma_ts_elect(acc1, a0 + 16 * u, b1 + off, idesc_o, (j > 0 || u > 0) ? 1u : 0u);  // acc1 += A0 B1
                }
            } else {  // B1 = G absent
#pragma unroll
                for (int u = 0; u < BC / 16; ++u) {
                    const uint64_t off = (uint64_t)((u * 16 * 128) >> 4);
                    const uint32_t acc = (j > 0 || u > 0) ? 1u : 0u;
                    ptx::mma_ts_elect(acc0, a0 + 16 * u, b0 + off, idesc_o, acc);   // acc0 += A0 B0
                    ptx::mma_ts_elect(acc1, a1 + 16 * u, b0 + off, idesc_o, acc);   // acc1 += A1 B0
                }
            }
            ptx::mma_commit_elect(bar(C::B_LEMPTY + g % SL));
            if (j == T - 1) ptx::mma_commit_elect(bar(C::B_FINAL));
            return true;
        };
        bool ok = true;
        if constexpr (NPAIR == 1) {
            // warp `wsel` owns the tiles g = wsel, wsel + 2, ...: S(g), then per tile outputs(g) and S(g + 2)
            int it = 0, j = wsel;  // of tile g
            while (j >= T) { j -= T; ++it; }
            if (wsel < G) ok = issue_scores(wsel, it, j);
            // The turn passes on after the whole batch (outputs(g), S(g + 2)): two batches queued at once
            // would share the pipe MMA by MMA, both would finish late and together, and the element-wise
            // work of the two buffers would then run back to back instead of under the other's MMAs.
            // Where the score MMAs belong to the next item they wait for its operands, which the element-wise
            // warps stage after their last tile: there the turn passes on before them, or the last output MMAs of
            // this item, and with them its epilogue, would wait for the next item's operands too.
            for (int g = wsel; ok && g < G; g += 2) {
                ok = issue_outputs(g, it, j);  // waits for the L tile, the operands and its turn
                const bool cross = j + 2 >= T;
                if (cross) {
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::turn_post(turn_addr, (uint32_t)g + 1u);
                }
                j += 2;
                while (j >= T) { j -= T; ++it; }
                if (ok && g + 2 < G) ok = issue_scores(g + 2, it, j);
                if (!cross) {
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::turn_post(turn_addr, (uint32_t)g + 1u);
                }
            }
        } else {
            if (wsel == 0) {  // one issuer: splitting these steps over two warps measured 1 to 2 % slower
                // One score buffer used in two phases.  Order on the tensor pipe:
                //   (S, Sd)(0), (D, X)(0), then per tile j: (S, Sd)(j+1) once the element-wise warps have read
                //   (S, Sd)(j) | outputs(j) once the operands W, dA are written | (D, X)(j+1), which overwrites them.
                const uint32_t dS = tb + C::COL_SCORE, dT = dS + BC, dD = dS + 2 * BC, dX = dS + 3 * BC;
                // One election per batch of MMAs and descriptors as 32-bit halves (see mma_ts_p): the issuing warp
                // shares its scheduler with four element-wise warps, and every instruction it saves per MMA shortens
                // the chain second pair -> phase B -> outputs -> second pair.  (DV and the forward, whose chains
                // are not bound by the issue, measured 2 to 4 % slower this way and keep the elected-lane form.)
                constexpr uint32_t HI_SW = HI_SW128;
                // [S | X0 Y1^T] = X0 [Y0 | Y1]^T, Sd += X1 Y0^T; X0, X1 in shared memory, Y0, Y1 in the L ring, all K-major.
                // `last`: the item's last tile; the shared-memory owner tiles are free once these MMAs are done
                auto issue_first_pair = [&](int g, bool last) {
                    const uint32_t el = ptx::elect_one();
                    const uint32_t st = l_stage(g);
#pragma unroll
                    for (int kk = 0; kk < KS; ++kk) {  // HZ: S = X0 Y0^T alone
                        const uint32_t ahi = kk < 4 ? HI_SW128 : HI_TAIL;
                        if (kk == 0) ptx::mma_ss_p<0>(el, dS, own_klo(own_base, kk), ahi, l_klo(st, kk), HI_SW128, HZ ? idesc_s : idesc_s2);
                        else ptx::mma_ss_p<1>(el, dS, own_klo(own_base, kk), ahi, l_klo(st, kk), HI_SW128, HZ ? idesc_s : idesc_s2);
                    }
                    if (!HZ) {
#pragma unroll
                        for (int kk = 0; kk < KS; ++kk)
                            ptx::mma_ss_p<1>(el, dT, own_klo(own_base + C::OWN_BYTES, kk), kk < 4 ? HI_SW128 : HI_TAIL, l_klo(st, kk), HI_SW128, idesc_s);
                    }
                    ptx::mma_commit_p(el, bar(C::B_SFULL + 0));
                    if (last) ptx::mma_commit_p(el, bar(C::B_OWNFREE));
                };
                // [D | X2 Y3^T] = X2 [Y2 | Y3]^T, X += X3 Y2^T; X2, X3 in tensor memory, Y2, Y3 in the E ring
                auto issue_second_pair = [&](int g) {
                    const uint32_t el = ptx::elect_one();
                    const uint32_t st = e_stage(g);
                    if (HZ) {
                        // X = G V^T alone.  DK: X2 Y3^T with X2 = V in tensor memory and Y3 = G the second tensor of the E
                        // stage; DQ: X3 Y2^T with X3 = G in tensor memory and Y2 = V the first tensor of the stage.
                        const uint32_t ya = MODE == BWD_DK ? st + BC * 128 : st, yt = st + 2 * BC * 128 + (MODE == BWD_DK ? BC * 16 : 0);
                        const uint32_t ax = MODE == BWD_DK ? ax0 : ax1;
#pragma unroll
                        for (int kk = 0; kk < KS; ++kk) {
                            const uint32_t lo = kk < 4 ? ptx::desc_lo(ya, 16) + 2u * kk : ptx::desc_lo(yt, 2 * BC * 16);
                            if (kk == 0) ptx::mma_ts_p<0>(el, dX, ax + 8 * kk, lo, kk < 4 ? HI_SW128 : HI_TAIL, idesc_s);
                            else ptx::mma_ts_p<1>(el, dX, ax + 8 * kk, lo, kk < 4 ? HI_SW128 : HI_TAIL, idesc_s);
                        }
                        ptx::mma_commit_p(el, bar(C::B_SFULL + 1));
                        ptx::mma_commit_p(el, bar(C::B_EEMPTY + g % SE));
                        return;
                    }
#pragma unroll
                    for (int kk = 0; kk < KS; ++kk) {
                        if (kk == 0) ptx::mma_ts_p<0>(el, dD, ax0 + 8 * kk, e_klo(st, kk), kk < 4 ? HI_SW128 : HI_TAIL, idesc_s2);
                        else ptx::mma_ts_p<1>(el, dD, ax0 + 8 * kk, e_klo(st, kk), kk < 4 ? HI_SW128 : HI_TAIL, idesc_s2);
                    }
                    // X3 Y2^T is zero when either factor is an absent cotangent: DK has Y2 = Hc, DQ has X3 = G
                    if (!(p.absent & (MODE == BWD_DK ? ABSENT_HC : ABSENT_G))) {
#pragma unroll
                        for (int kk = 0; kk < KS; ++kk) ptx::mma_ts_p<1>(el, dX, ax1 + 8 * kk, e_klo(st, kk), kk < 4 ? HI_SW128 : HI_TAIL, idesc_s);
                    }
                    ptx::mma_commit_p(el, bar(C::B_SFULL + 1));
                    ptx::mma_commit_p(el, bar(C::B_EEMPTY + g % SE));
                };
                for (int it = 0; ok && it < n_it; ++it) {
                    const int g0 = it * T;
                    // the item's owner operands: X0, X1 in tensor memory, X2, X3 in shared memory
                    ok = ptx::mbar_wait_warp(bar(C::B_QREADY + (it & 1)), (it >> 1) & 1, abort_flag, BWD_WAIT_LIMIT_NS);
                    if (ok) ok = ptx::mbar_wait_warp(bar(C::B_OWNER), it & 1, abort_flag, BWD_WAIT_LIMIT_NS);
                    // (S, Sd) of the tile before, the last of the item before, read by all element-wise warps
                    if (ok && it > 0) ok = ptx::mbar_wait_warp(bar(C::B_PREADY + 1), (g0 - 1) & 1, abort_flag, BWD_WAIT_LIMIT_NS);
                    if (ok) ok = ptx::mbar_wait_warp(bar(C::B_LFULL + g0 % SL), (g0 / SL) & 1, abort_flag, BWD_WAIT_LIMIT_NS);
                    if (ok) ok = ptx::mbar_wait_warp(bar(C::B_EFULL + g0 % SE), (g0 / SE) & 1, abort_flag, BWD_WAIT_LIMIT_NS);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    issue_first_pair(g0, T == 1);
                    issue_second_pair(g0);
                    for (int j = 0; ok && j < T; ++j) {
                        const int g = g0 + j;
                        if (j + 1 < T) {
                            const int gn = g + 1;
                            // (S, Sd)(g) read by all element-wise warps, and the tiles of g+1 loaded
                            const bool ready = ptx::mbar_test3_warp(bar(C::B_PREADY + 1), g & 1, bar(C::B_LFULL + gn % SL), (gn / SL) & 1,
                                                                    bar(C::B_EFULL + gn % SE), (gn / SE) & 1);
                            if (!ready) {
                                ok = ptx::mbar_wait_warp(bar(C::B_PREADY + 1), g & 1, abort_flag, BWD_WAIT_LIMIT_NS);
                                if (ok) ok = ptx::mbar_wait_warp(bar(C::B_LFULL + gn % SL), (gn / SL) & 1, abort_flag, BWD_WAIT_LIMIT_NS);
                                if (ok) ok = ptx::mbar_wait_warp(bar(C::B_EFULL + gn % SE), (gn / SE) & 1, abort_flag, BWD_WAIT_LIMIT_NS);
                                if (!ok) break;
                            }
                            ptx::tc_fence_after_sync();
                            issue_first_pair(gn, j + 2 == T);
                        }
                        // outputs(g): acc0 += W B0, acc1 += dA B0 + W B1 with the operands in the D and X columns
                        ok = ptx::mbar_wait_warp(bar(C::B_PREADY + 0), g & 1, abort_flag, BWD_WAIT_LIMIT_NS);
                        // the first tile of an item overwrites the accumulators: the element-wise warps have read them
                        if (ok && j == 0 && it > 0) ok = ptx::mbar_wait_warp(bar(C::B_ACCFREE + ((it - 1) & 1)), ((it - 1) >> 1) & 1, abort_flag, BWD_WAIT_LIMIT_NS);
                        if (!ok) break;
                        ptx::tc_fence_after_sync();
                        {
                            const uint32_t el = ptx::elect_one();
                            const uint32_t b0 = l_nlo(l_stage(g), 0, 0), b1 = l_nlo(l_stage(g), 1, 0);  // MN-major B
                            const bool hasW = !HZ && !(p.absent & ABSENT_HC);
                            const uint32_t acc0 = tb + C::COL_ACC0, acc1 = tb + C::COL_ACC1;
                            // with Hc absent W is exactly zero (D = 0 from zero operands, Sigma1 = 0): its MMAs are skipped.
                            // One uniform branch around the unrolled loops, none inside them.
                            if (hasW) {
#pragma unroll
                                for (int u = 0; u < BC / 16; ++u) {
                                    const uint32_t off = (uint32_t)((u * 16 * 128) >> 4);
                                    if (u == 0 && j == 0) {
                                        ptx::mma_ts_p<0>(el, acc0, dD + 16 * u, b0 + off, HI_SW, idesc_o);
                                        ptx::mma_ts_p<0>(el, acc1, dX + 16 * u, b0 + off, HI_SW, idesc_o);
                                    } else {
                                        ptx::mma_ts_p<1>(el, acc0, dD + 16 * u, b0 + off, HI_SW, idesc_o);
                                        ptx::mma_ts_p<1>(el, acc1, dX + 16 * u, b0 + off, HI_SW, idesc_o);
                                    }
                                    ptx::mma_ts_p<1>(el, acc1, dD + 16 * u, b1 + off, HI_SW, idesc_o);
                                }
                            } else {
#pragma unroll
                                for (int u = 0; u < BC / 16; ++u) {
                                    const uint32_t off = (uint32_t)((u * 16 * 128) >> 4);
                                    if (u == 0 && j == 0) ptx::mma_ts_p<0>(el, acc1, dX + 16 * u, b0 + off, HI_SW, idesc_o);
                                    else ptx::mma_ts_p<1>(el, acc1, dX + 16 * u, b0 + off, HI_SW, idesc_o);
                                }
                            }
                            ptx::mma_commit_p(el, bar(C::B_LEMPTY + g % SL));
                            if (j == T - 1) ptx::mma_commit_p(el, bar(C::B_FINAL));
                        }
                        if (j + 1 < T) issue_second_pair(g + 1);
                    }
                }
            }
        }
    } else {
        bwd_elementwise<MODE, DP, HZ>(p, tmem_base, bar0, abort_flag, stats, warp - 4, lane, items, row_tiles, T);
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
    // DK and DQ start while the pass before them still runs (programmatic dependent launch) and read nothing it
    // writes; they must still not complete before it, or completion of the last pass would not imply that the
    // gradients of the earlier ones are written.  (No effect on a launch without the attribute.)
    if (MODE != BWD_DV && threadIdx.x == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
}

}  // namespace tvm_attn
