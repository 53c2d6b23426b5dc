// Tensor-core (tcgen05 + TMEM + TMA) kernel for attention with a Jacobian-vector product, forward
// and backward, on sm_100a.
//
// One kernel skeleton serves four passes, because carrying a tangent next to a primal is
// dual-number arithmetic and every product of the method has the same shape
//     (a + eps b)(c + eps d) = ac + eps (bc + ad).
// A CTA owns 128 "owner" rows of one head and streams the other side in tiles of BC rows:
//
//   pass   owner rows  stream rows  score accumulators (128 x BC, fp32 in TMEM)        operands A0, A1 (bf16)   acc0, acc1 (128 x d)
//   FWD    queries     keys         S = Q K^T, Sd = tQ K^T + Q tK^T                       P~, P~*T                 O~, R
//   DV     keys        queries      S^T, Sd^T                                             P^T, (P*Nn)^T            dtV, dV
//   DK     keys        queries      S^T, Sd^T, D^T = V Hc^T, X^T = V G^T + tV Hc^T        W^T, dA^T                dtK/alpha, dK/alpha
//   DQ     queries     keys         S, Sd, D = Hc V^T, X = G V^T + Hc tV^T                W, dA                    dtQ/alpha, dQ/alpha
//
// with, per score pair (X0, X1 owner tiles; Y0, Y1 stream tiles):  S = X0 Y0^T,  Sd = X1 Y0^T + X0 Y1^T,
// and for the outputs (B0, B1 stream tiles):  acc0 += A0 B0,  acc1 += A1 B0 + A0 B1.
// (Forward: App. C Eq. "sdpa" and the definitions under "Step 1"; DV: step 6; DK: steps 2 and 4;
// DQ: steps 3 and 5; each with the standard attention backward for dO added in.)
//
// Roles (384 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warp 2 = loader
// of per-query statistics for the transposed passes, warp 3 idle, warps 4-11 = element-wise warps
// (two per TMEM lane quadrant).  Score accumulators are double-buffered in TMEM so that the MMAs
// of tile j+1 run while tile j is in the element-wise stage; the bf16 operands A0/A1 are written
// back into the columns of the score accumulators they came from and consumed from TMEM.
//
// Shared-memory tiles are 128-byte-swizzled boxes of 64 bf16 columns ("atoms"); a head dim above 64
// uses two atoms per row, the second zero-filled beyond d by TMA, so d = 72 runs as 80.
// Every wait on an mbarrier is bounded; when one gives up the block records a time-out status and
// all roles leave their loops.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "sm100_ptx.cuh"

namespace tvm_attn {

enum : int { MODE_FWD = 0, MODE_DV = 1, MODE_DK = 2, MODE_DQ = 3 };

constexpr int TC_THREADS = 384;
constexpr int TC_OWN_ROWS = 128;
constexpr int TC_STATS_STAGES = 4;
constexpr uint64_t TC_WAIT_LIMIT_NS = 200ull * 1000ull * 1000ull;  // 0.2 s per wait
constexpr float TC_RESCALE_THRESHOLD = 8.0f;  // log2 units: accumulators are rescaled only past this
constexpr float TC_CENTER_DELTA = 3.0f;       // the centre of the tangent weights moves only past this

struct TcParams {
    int N, d, dp, BH;
    float alpha;      // softmax scale
    float c2;         // alpha * log2(e)
    float out_scale;  // factor applied to acc0/acc1 in the epilogue of the backward passes
    void* out0;       // acc0 destination: O | dtV | dtK | dtQ
    void* out1;       // acc1 destination: tO | dV | dK | dQ
    float* lse_out;   // FWD
    float* mu_out;    // FWD
    const float* lse; // backward passes
    const float* mu;
    const float* sig1;
    const float* cvec;
    int* status;      // device status word; non-zero makes the kernel a no-op
};

template <int MODE, int NA>
struct TcCfg {
    static constexpr int NPAIR = (MODE == MODE_FWD || MODE == MODE_DV) ? 1 : 2;
    static constexpr int NOWN = 2 * NPAIR;
    static constexpr int BC = NPAIR == 1 ? 64 : 32;
    static constexpr bool TRANSPOSED = (MODE == MODE_DV || MODE == MODE_DK);
    static constexpr int SE = NA == 1 ? 3 : 2;
    static constexpr int SL = NA == 1 ? (NPAIR == 1 ? 3 : 4) : (NPAIR == 1 ? 2 : 3);
    static constexpr int OWN_BYTES = NA * TC_OWN_ROWS * 128;
    static constexpr int ST_BYTES = NA * BC * 128;
    static constexpr int TILE_BYTES = NOWN * OWN_BYTES + (SE + SL) * 2 * ST_BYTES;
    // barrier slots
    static constexpr int B_OWNER = 0;
    static constexpr int B_EFULL = 1;
    static constexpr int B_EEMPTY = B_EFULL + SE;
    static constexpr int B_LFULL = B_EEMPTY + SE;
    static constexpr int B_LEMPTY = B_LFULL + SL;
    static constexpr int B_SFULL = B_LEMPTY + SL;
    static constexpr int B_PREADY = B_SFULL + 2;
    static constexpr int B_OUTDONE = B_PREADY + 2;
    static constexpr int B_FINAL = B_OUTDONE + 1;
    static constexpr int B_STFULL = B_FINAL + 1;
    static constexpr int B_STEMPTY = B_STFULL + TC_STATS_STAGES;
    static constexpr int B_XCHG = B_STEMPTY + TC_STATS_STAGES;
    static constexpr int NBARS = B_XCHG + 4;
    static constexpr int MISC_BYTES = 8 * 64 /*barriers*/ + 64 /*tmem ptr, abort*/ +
                                      TC_STATS_STAGES * 4 * 64 * 4 /*stats*/ + 2 * 2 * 2 * 128 * 4 /*xchg*/;
    static constexpr int SMEM_BYTES = TILE_BYTES + MISC_BYTES + 1024 /*alignment slack*/;
    static_assert(NBARS <= 64, "barrier table too small");
    // TMEM columns
    static constexpr int COL_ACC0 = 0, COL_ACC1 = 128, COL_SCORE = 256, SCORE_BUF_COLS = 2 * NPAIR * BC;
    static_assert(COL_SCORE + 2 * SCORE_BUF_COLS <= 512, "TMEM over-subscribed");
};


// ---- MMA issue helpers.  One thread issues every tcgen05.mma of a CTA, so the instruction count per
// MMA matters: descriptors are built once per tile and advanced by compile-time offsets.

// One GEMM  D[128 x ROWS_B] (+)= A[128 x 16*KS] * B[ROWS_B x 16*KS]^T  from K-major tiles whose
// 64-column atoms are `rows * 128` bytes apart; k-step kk lives 32*(kk%4) bytes into atom kk/4.
template <int KS, int ROWS_B>
__device__ __forceinline__ void issue_kmajor_gemm(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, bool accumulate) {
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
        const uint64_t off_a = (uint64_t)(((kk >> 2) * TC_OWN_ROWS * 128 + (kk & 3) * 32) >> 4);
        const uint64_t off_b = (uint64_t)(((kk >> 2) * ROWS_B * 128 + (kk & 3) * 32) >> 4);
        ptx::mma_ss_elect(d, a + off_a, b + off_b, idesc, (accumulate || kk > 0) ? 1u : 0u);
    }
}

// Score MMAs of one tile:  S = X0 Y0^T,  Sd = X1 Y0^T + X0 Y1^T  per score pair.
template <int KS, int NPAIR, int BC>
__device__ __forceinline__ void issue_score_mmas(const uint64_t* xd, const uint64_t* yd, uint32_t dbase, uint32_t idesc) {
#pragma unroll
    for (int pr = 0; pr < NPAIR; ++pr) {
        const uint32_t dS = dbase + 2 * pr * BC, dT = dS + BC;
        issue_kmajor_gemm<KS, BC>(dS, xd[2 * pr], yd[2 * pr], idesc, false);
        issue_kmajor_gemm<KS, BC>(dT, xd[2 * pr + 1], yd[2 * pr], idesc, false);
        issue_kmajor_gemm<KS, BC>(dT, xd[2 * pr], yd[2 * pr + 1], idesc, true);
    }
}

template <int NPAIR, int BC>
__device__ __forceinline__ void issue_score_mmas_dyn(int ksteps, const uint64_t* xd, const uint64_t* yd, uint32_t dbase,
                                                     uint32_t idesc) {
    switch (ksteps) {
        case 1: issue_score_mmas<1, NPAIR, BC>(xd, yd, dbase, idesc); break;
        case 2: issue_score_mmas<2, NPAIR, BC>(xd, yd, dbase, idesc); break;
        case 3: issue_score_mmas<3, NPAIR, BC>(xd, yd, dbase, idesc); break;
        case 4: issue_score_mmas<4, NPAIR, BC>(xd, yd, dbase, idesc); break;
        case 5: issue_score_mmas<5, NPAIR, BC>(xd, yd, dbase, idesc); break;
        case 6: issue_score_mmas<6, NPAIR, BC>(xd, yd, dbase, idesc); break;
        case 7: issue_score_mmas<7, NPAIR, BC>(xd, yd, dbase, idesc); break;
        default: issue_score_mmas<8, NPAIR, BC>(xd, yd, dbase, idesc); break;
    }
}

// Output MMAs of one tile:  acc0 += A0 B0,  acc1 += A1 B0 + A0 B1  with A from TMEM (operand of
// k-step u at column 16u of its score accumulator) and B MN-major (k-step u = 16 stream rows = 2048 B).
template <int BC>
__device__ __forceinline__ void issue_output_mmas(uint32_t acc0, uint32_t acc1, uint32_t a0, uint32_t a1, uint64_t b0,
                                                  uint64_t b1, uint32_t idesc, bool accumulate) {
#pragma unroll
    for (int u = 0; u < BC / 16; ++u) {
        const uint64_t off = (uint64_t)((u * 16 * 128) >> 4);
        const uint32_t acc = (accumulate || u > 0) ? 1u : 0u;
        ptx::mma_ts_elect(acc0, a0 + 16 * u, b0 + off, idesc, acc);
        ptx::mma_ts_elect(acc1, a1 + 16 * u, b0 + off, idesc, acc);
        ptx::mma_ts_elect(acc1, a0 + 16 * u, b1 + off, idesc, 1u);
    }
}

template <int MODE, int NA>
__global__ void __launch_bounds__(TC_THREADS, 1)
dual_attn_kernel(const __grid_constant__ CUtensorMap tm_own0, const __grid_constant__ CUtensorMap tm_own1,
                 const __grid_constant__ CUtensorMap tm_own2, const __grid_constant__ CUtensorMap tm_own3,
                 const __grid_constant__ CUtensorMap tm_st0, const __grid_constant__ CUtensorMap tm_st1,
                 const __grid_constant__ CUtensorMap tm_st2, const __grid_constant__ CUtensorMap tm_st3,
                 const TcParams p) {
    using C = TcCfg<MODE, NA>;
    constexpr int BC = C::BC, NPAIR = C::NPAIR, SE = C::SE, SL = C::SL;
    if (*reinterpret_cast<volatile int*>(p.status) != 0) return;  // an earlier kernel timed out

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t own_base = ptx::smem_u32(smem);
    const uint32_t e_base = own_base + C::NOWN * C::OWN_BYTES;
    const uint32_t l_base = e_base + SE * 2 * C::ST_BYTES;
    uint8_t* misc = smem + C::TILE_BYTES;
    const uint32_t bar0 = ptx::smem_u32(misc);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 8 * 64);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 8 * 64 + 16);
    float* stats = reinterpret_cast<float*>(misc + 8 * 64 + 64);  // [stage][4][64]
    float* xchg = stats + TC_STATS_STAGES * 4 * 64;               // [parity][half][value][128]
    auto bar = [&](int i) -> uint32_t { return bar0 + 8u * static_cast<uint32_t>(i); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int own_tiles = (p.N + TC_OWN_ROWS - 1) / TC_OWN_ROWS;
    const int bh = blockIdx.x / own_tiles;
    const int row0 = (blockIdx.x - bh * own_tiles) * TC_OWN_ROWS;
    const int T = (p.N + BC - 1) / BC;  // stream tiles
    const int ksteps = p.dp >> 4;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        ptx::mbar_init(bar(C::B_OWNER), 1);
        for (int s = 0; s < SE; ++s) { ptx::mbar_init(bar(C::B_EFULL + s), 1); ptx::mbar_init(bar(C::B_EEMPTY + s), 1); }
        for (int s = 0; s < SL; ++s) { ptx::mbar_init(bar(C::B_LFULL + s), 1); ptx::mbar_init(bar(C::B_LEMPTY + s), 1); }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(bar(C::B_SFULL + b), 1);
            ptx::mbar_init(bar(C::B_PREADY + b), MODE == MODE_FWD ? 256 : 128);
        }
        ptx::mbar_init(bar(C::B_OUTDONE), 1);
        ptx::mbar_init(bar(C::B_FINAL), 1);
        for (int s = 0; s < TC_STATS_STAGES; ++s) {
            ptx::mbar_init(bar(C::B_STFULL + s), 32);
            ptx::mbar_init(bar(C::B_STEMPTY + s), 128);
        }
        for (int q = 0; q < 4; ++q) ptx::mbar_init(bar(C::B_XCHG + q), 64);
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(tmem_slot), 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    // Which stream tensors travel in the early-released ring (E) and the late-released ring (L).
    // One score pair: E = {Y0, Y1} (score operands), L = {B0, B1} (output operands).
    // Two score pairs: L = {Y0, Y1} (also the output operands B0, B1), E = {Y2, Y3}.
    constexpr int E_FIRST = NPAIR == 1 ? 0 : 2;
    constexpr int L_FIRST = NPAIR == 1 ? 2 : 0;
    auto stream_addr = [&](int t, int j) -> uint32_t {  // smem address of stream tile t (0..3) of iteration j
        const bool in_e = (t >= E_FIRST) && (t < E_FIRST + 2);
        return in_e ? e_base + ((j % SE) * 2 + (t - E_FIRST)) * C::ST_BYTES
                    : l_base + ((j % SL) * 2 + (t - L_FIRST)) * C::ST_BYTES;
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const CUtensorMap* own_maps[4] = {&tm_own0, &tm_own1, &tm_own2, &tm_own3};
            const CUtensorMap* st_maps[4] = {&tm_st0, &tm_st1, &tm_st2, &tm_st3};
            ptx::mbar_arrive_expect_tx(bar(C::B_OWNER), C::NOWN * C::OWN_BYTES);
            for (int t = 0; t < C::NOWN; ++t)
                for (int a = 0; a < NA; ++a)
                    ptx::tma_load_3d(own_base + t * C::OWN_BYTES + a * TC_OWN_ROWS * 128, own_maps[t],
                                     bar(C::B_OWNER), a * 64, row0, bh);
            for (int j = 0; j < T; ++j) {
                // the ring whose tiles the score MMAs of a two-pair pass need first goes first
                for (int ring = 0; ring < 2; ++ring) {
                    const bool is_e = (ring == 0);
                    const int S = is_e ? SE : SL;
                    const int s = j % S, ph = (j / S) & 1;
                    const int full = (is_e ? C::B_EFULL : C::B_LFULL) + s;
                    const int empty = (is_e ? C::B_EEMPTY : C::B_LEMPTY) + s;
                    if (!ptx::mbar_wait(bar(empty), ph ^ 1, abort_flag, TC_WAIT_LIMIT_NS)) goto producer_done;
                    ptx::mbar_arrive_expect_tx(bar(full), 2 * C::ST_BYTES);
                    const int first = is_e ? E_FIRST : L_FIRST;
                    for (int t = first; t < first + 2; ++t)
                        for (int a = 0; a < NA; ++a)
                            ptx::tma_load_3d(stream_addr(t, j) + a * BC * 128, st_maps[t], bar(full), a * 64, j * BC, bh);
                }
            }
        producer_done:;
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        {   // the whole warp runs the loop; one elected lane issues (see mma_ts_elect)
            const uint32_t idesc_s = ptx::idesc_bf16_f32(128, BC, 0, 0);
            const uint32_t idesc_o = ptx::idesc_bf16_f32(128, p.dp, 0, 1);
            // descriptors of the resident owner tiles (K-major) never change
            uint64_t xd[4];
#pragma unroll
            for (int t = 0; t < 4; ++t)
                xd[t] = ptx::smem_desc_sw128(own_base + (t < C::NOWN ? t : 0) * C::OWN_BYTES, 16, 1024);
            bool ok = ptx::mbar_wait_warp(bar(C::B_OWNER), 0, abort_flag, TC_WAIT_LIMIT_NS);
            auto issue_scores = [&](int j) -> bool {
                const int b = j & 1;
                if (!ptx::mbar_wait_warp(bar(C::B_EFULL + j % SE), (j / SE) & 1, abort_flag, TC_WAIT_LIMIT_NS)) return false;
                if (NPAIR == 2)
                    if (!ptx::mbar_wait_warp(bar(C::B_LFULL + j % SL), (j / SL) & 1, abort_flag, TC_WAIT_LIMIT_NS)) return false;
                ptx::tc_fence_after_sync();
                uint64_t yd[4];
#pragma unroll
                for (int t = 0; t < 2 * NPAIR; ++t) yd[t] = ptx::smem_desc_sw128(stream_addr(t, j), 16, 1024);
                issue_score_mmas_dyn<NPAIR, BC>(ksteps, xd, yd, tmem_base + C::COL_SCORE + b * C::SCORE_BUF_COLS, idesc_s);
                ptx::mma_commit_elect(bar(C::B_SFULL + b));
                ptx::mma_commit_elect(bar(C::B_EEMPTY + j % SE));
                return true;
            };
            auto issue_outputs = [&](int j) -> bool {
                const int b = j & 1;
                if (NPAIR == 1)
                    if (!ptx::mbar_wait_warp(bar(C::B_LFULL + j % SL), (j / SL) & 1, abort_flag, TC_WAIT_LIMIT_NS)) return false;
                if (!ptx::mbar_wait_warp(bar(C::B_PREADY + b), (j >> 1) & 1, abort_flag, TC_WAIT_LIMIT_NS)) return false;
                ptx::tc_fence_after_sync();
                const uint32_t a0 = tmem_base + C::COL_SCORE + b * C::SCORE_BUF_COLS, a1 = a0 + BC;
                // MN-major: atoms of 64 d-columns are BC*128 bytes apart, 8-row groups 1024 bytes apart
                const uint64_t b0 = ptx::smem_desc_sw128(stream_addr(L_FIRST, j), BC * 128, 1024);
                const uint64_t b1 = ptx::smem_desc_sw128(stream_addr(L_FIRST + 1, j), BC * 128, 1024);
                issue_output_mmas<BC>(tmem_base + C::COL_ACC0, tmem_base + C::COL_ACC1, a0, a1, b0, b1, idesc_o, j > 0);
                ptx::mma_commit_elect(bar(C::B_LEMPTY + j % SL));
                ptx::mma_commit_elect(bar(C::B_OUTDONE));
                if (j == T - 1) ptx::mma_commit_elect(bar(C::B_FINAL));
                return true;
            };
            if (ok) ok = issue_scores(0);
            for (int j = 0; ok && j < T; ++j) {
                if (j + 1 < T) ok = issue_scores(j + 1);
                if (ok) ok = issue_outputs(j);
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ per-query statistics (transposed passes)
        if (C::TRANSPOSED) {
            const size_t srow = (size_t)bh * p.N;
            for (int j = 0; j < T; ++j) {
                const int s = j % TC_STATS_STAGES, ph = (j / TC_STATS_STAGES) & 1;
                if (!ptx::mbar_wait(bar(C::B_STEMPTY + s), ph ^ 1, abort_flag, TC_WAIT_LIMIT_NS)) break;
                float* st = stats + s * 4 * 64;
                for (int c = lane; c < BC; c += 32) {
                    const int i = j * BC + c;
                    const bool v = i < p.N;
                    st[0 * 64 + c] = v ? p.lse[srow + i] * 1.4426950408889634f : CUDART_INF_F;
                    st[1 * 64 + c] = v ? p.mu[srow + i] : 0.f;
                    if (MODE == MODE_DK) {
                        st[2 * 64 + c] = v ? p.sig1[srow + i] : 0.f;
                        st[3 * 64 + c] = v ? p.cvec[srow + i] : 0.f;
                    }
                }
                ptx::mbar_arrive(bar(C::B_STFULL + s));
            }
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ element-wise warps
        const int g = (warp - 4) >> 2;  // warpgroup 0/1
        const int q = warp & 3;         // TMEM lane quadrant
        const int row = q * 32 + lane;  // owner row inside the CTA tile
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
        const bool row_valid = row0 + row < p.N;
        bool ok = true;

        if (MODE == MODE_FWD) {
            // Online softmax with two refinements.  (1) The reference maximum m_ref follows the true
            // running maximum lazily: accumulators are rescaled only when a tile maximum exceeds it by
            // more than TC_RESCALE_THRESHOLD (log2 units).  (2) The tangent weights are centred,
            // T - c, with c the value of T at the row's running arg-max key, so that the bf16 rounding
            // of P~*(T - c) is small where P~ is large; tO = R'/l - (mu - c) O with R' = sum P~ (T - c) V.
            // c moves only when a new row maximum arrives whose T differs from c by more than
            // TC_CENTER_DELTA; then R' += (c_old - c_new) O~ keeps the accumulators consistent.
            float m_ref = -CUDART_INF_F, m_true = -CUDART_INF_F, cen = 0.f, l = 0.f, mt = 0.f;
            const int col0 = g * 32;
            for (int j = 0; j < T; ++j) {
                const int b = j & 1;
                if (!ptx::mbar_wait(bar(C::B_SFULL + b), (j >> 1) & 1, abort_flag, TC_WAIT_LIMIT_NS)) { ok = false; break; }
                ptx::tc_fence_after_sync();
                const uint32_t sbase = lane_addr + C::COL_SCORE + b * C::SCORE_BUF_COLS;
                uint32_t s[32], ts[32];
                ptx::tmem_ld16(sbase + col0, s);
                ptx::tmem_ld16(sbase + col0 + 16, s + 16);
                ptx::tmem_ld16(sbase + BC + col0, ts);
                ptx::tmem_ld16(sbase + BC + col0 + 16, ts + 16);
                ptx::tmem_wait_ld();
                const int nvalid = p.N - j * BC - col0;  // columns of this half that are real keys
                if (nvalid < 32) {
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (c >= nvalid) s[c] = __float_as_uint(-CUDART_INF_F);
                }
                // maximum of this half and the tangent score at that key (pairwise tree: short dependency chain)
                float mx, tw;
                {
                    float vm[16], vt[16];
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        const float a = __uint_as_float(s[2 * c]), b2 = __uint_as_float(s[2 * c + 1]);
                        const bool gt = b2 > a;
                        vm[c] = gt ? b2 : a;
                        vt[c] = gt ? __uint_as_float(ts[2 * c + 1]) : __uint_as_float(ts[2 * c]);
                    }
#pragma unroll
                    for (int w = 8; w >= 1; w >>= 1) {
#pragma unroll
                        for (int c = 0; c < w; ++c) {
                            const bool gt = vm[c + w] > vm[c];
                            vm[c] = gt ? vm[c + w] : vm[c];
                            vt[c] = gt ? vt[c + w] : vt[c];
                        }
                    }
                    mx = vm[0];
                    tw = vt[0];
                }
                mx *= p.c2;
                tw *= p.alpha;
                // the two threads that share a row (one per warpgroup) agree on the tile maximum
                float* xslot = xchg + (j & 1) * 512;
                xslot[g * 256 + row] = mx;
                xslot[g * 256 + 128 + row] = tw;
                ptx::mbar_arrive(bar(C::B_XCHG + q));
                if (!ptx::mbar_wait(bar(C::B_XCHG + q), j & 1, abort_flag, TC_WAIT_LIMIT_NS)) { ok = false; break; }
                {
                    const float omx = xslot[(g ^ 1) * 256 + row], otw = xslot[(g ^ 1) * 256 + 128 + row];
                    const bool other_wins = (g == 0) ? (omx > mx) : (omx >= mx);  // ties go to half 0
                    tw = other_wins ? otw : tw;
                    mx = fmaxf(mx, omx);
                }
                const bool need_scale = mx > m_ref + TC_RESCALE_THRESHOLD;
                const bool need_cen = (mx > m_true) && (j == 0 || fabsf(tw - cen) > TC_CENTER_DELTA);
                m_true = fmaxf(m_true, mx);
                if (__any_sync(0xffffffffu, need_scale || need_cen)) {
                    const float scale = need_scale ? ptx::ex2(m_ref - mx) : 1.0f;
                    const float fix = need_cen ? cen - tw : 0.f;
                    if (need_scale) m_ref = mx;
                    if (need_cen) cen = tw;
                    mt = scale * fmaf(fix, l, mt);
                    l *= scale;
                    if (j > 0) {
                        // accumulators must be at rest: the output MMAs of tile j-1 have completed
                        if (!ptx::mbar_wait(bar(C::B_OUTDONE), (j - 1) & 1, abort_flag, TC_WAIT_LIMIT_NS)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        for (int ch = g; ch < ksteps; ch += 2) {
                            uint32_t o[16], r[16];
                            ptx::tmem_ld16(lane_addr + C::COL_ACC0 + 16 * ch, o);
                            ptx::tmem_ld16(lane_addr + C::COL_ACC1 + 16 * ch, r);
                            ptx::tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < 16; ++c) {
                                const float ov = __uint_as_float(o[c]);
                                r[c] = __float_as_uint(scale * fmaf(fix, ov, __uint_as_float(r[c])));
                                o[c] = __float_as_uint(scale * ov);
                            }
                            ptx::tmem_st16(lane_addr + C::COL_ACC0 + 16 * ch, o);
                            ptx::tmem_st16(lane_addr + C::COL_ACC1 + 16 * ch, r);
                        }
                    }
                }
                uint32_t pp[16], ppt[16];
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                    const float p0 = ptx::ex2(fmaf(__uint_as_float(s[c]), p.c2, -m_ref));
                    const float p1 = ptx::ex2(fmaf(__uint_as_float(s[c + 1]), p.c2, -m_ref));
                    const float t0 = p0 * fmaf(p.alpha, __uint_as_float(ts[c]), -cen);
                    const float t1 = p1 * fmaf(p.alpha, __uint_as_float(ts[c + 1]), -cen);
                    l += p0 + p1;
                    mt += t0 + t1;
                    pp[c >> 1] = ptx::pack_bf16(p0, p1);
                    ppt[c >> 1] = ptx::pack_bf16(t0, t1);
                }
                // operand of k-step kk (16 keys) sits at column 16*kk of the accumulator it replaces
                ptx::tmem_st8(sbase + col0, pp);
                ptx::tmem_st8(sbase + col0 + 16, pp + 8);
                ptx::tmem_st8(sbase + BC + col0, ppt);
                ptx::tmem_st8(sbase + BC + col0 + 16, ppt + 8);
                ptx::tmem_wait_st();
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive(bar(C::B_PREADY + b));
            }
            // ---- epilogue: O = O~/l, mu - c = mt/l, tO = R'/l - (mu - c) O, lse = ln2 (m_ref + log2 l)
            if (ok) ok = ptx::mbar_wait(bar(C::B_FINAL), 0, abort_flag, TC_WAIT_LIMIT_NS);
            if (ok) {
                ptx::tc_fence_after_sync();
                float* xslot = xchg + (T & 1) * 512;
                xslot[g * 256 + row] = l;
                xslot[g * 256 + 128 + row] = mt;
                ptx::mbar_arrive(bar(C::B_XCHG + q));
                ok = ptx::mbar_wait(bar(C::B_XCHG + q), T & 1, abort_flag, TC_WAIT_LIMIT_NS);
            }
            if (ok) {
                const float* xslot = xchg + (T & 1) * 512;
                l += xslot[(g ^ 1) * 256 + row];
                mt += xslot[(g ^ 1) * 256 + 128 + row];
                const float inv = 1.0f / l;
                const float mun = mt * inv;
                __nv_bfloat16* o_ptr = reinterpret_cast<__nv_bfloat16*>(p.out0) + ((size_t)bh * p.N + row0 + row) * p.d;
                __nv_bfloat16* t_ptr = reinterpret_cast<__nv_bfloat16*>(p.out1) + ((size_t)bh * p.N + row0 + row) * p.d;
                for (int ch = g; ch < ksteps; ch += 2) {
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
                if (g == 0 && row_valid) {
                    p.lse_out[(size_t)bh * p.N + row0 + row] = (m_ref + log2f(l)) * 0.6931471805599453f;
                    p.mu_out[(size_t)bh * p.N + row0 + row] = cen + mun;
                }
            }
        } else {
            // ---- backward passes: warpgroup g takes the tiles j = g, g+2, ... (score buffer g)
            float r_lse2 = CUDART_INF_F, r_mu = 0.f, r_s1 = 0.f, r_cv = 0.f;
            if (MODE == MODE_DQ && row_valid) {
                const size_t i = (size_t)bh * p.N + row0 + row;
                r_lse2 = p.lse[i] * 1.4426950408889634f;
                r_mu = p.mu[i];
                r_s1 = p.sig1[i];
                r_cv = p.cvec[i];
            }
            for (int j = g; j < T; j += 2) {
                const int b = j & 1;
                if (!ptx::mbar_wait(bar(C::B_SFULL + b), (j >> 1) & 1, abort_flag, TC_WAIT_LIMIT_NS)) { ok = false; break; }
                const float* st = stats + (j % TC_STATS_STAGES) * 4 * 64;
                if (C::TRANSPOSED)
                    if (!ptx::mbar_wait(bar(C::B_STFULL + j % TC_STATS_STAGES), (j / TC_STATS_STAGES) & 1, abort_flag,
                                        TC_WAIT_LIMIT_NS)) { ok = false; break; }
                ptx::tc_fence_after_sync();
                const uint32_t sbase = lane_addr + C::COL_SCORE + b * C::SCORE_BUF_COLS;
                for (int u = 0; u < BC / 16; ++u) {
                    uint32_t s1[16], s2[16], s3[16], s4[16];
                    ptx::tmem_ld16(sbase + 16 * u, s1);
                    ptx::tmem_ld16(sbase + BC + 16 * u, s2);
                    if (NPAIR == 2) {
                        ptx::tmem_ld16(sbase + 2 * BC + 16 * u, s3);
                        ptx::tmem_ld16(sbase + 3 * BC + 16 * u, s4);
                    }
                    ptx::tmem_wait_ld();
                    uint32_t pa0[8], pa1[8];
#pragma unroll
                    for (int c = 0; c < 16; c += 2) {
                        float a0[2], a1[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int col = 16 * u + c + e;
                            float lse2, mu, sg = 0.f, cv = 0.f;
                            if (C::TRANSPOSED) {
                                lse2 = st[col]; mu = st[64 + col];
                                if (MODE == MODE_DK) { sg = st[128 + col]; cv = st[192 + col]; }
                            } else {
                                lse2 = (j * BC + col < p.N) ? r_lse2 : CUDART_INF_F;  // keys beyond N: P = 0
                                mu = r_mu; sg = r_s1; cv = r_cv;
                            }
                            const float P = ptx::ex2(fmaf(__uint_as_float(s1[c + e]), p.c2, -lse2));
                            const float Nn = fmaf(p.alpha, __uint_as_float(s2[c + e]), -mu);
                            if (MODE == MODE_DV) {
                                a0[e] = P;
                                a1[e] = P * Nn;
                            } else {
                                const float W = P * (__uint_as_float(s3[c + e]) - sg);
                                a0[e] = W;
                                a1[e] = fmaf(P, __uint_as_float(s4[c + e]) - cv, W * Nn);
                            }
                        }
                        pa0[c >> 1] = ptx::pack_bf16(a0[0], a0[1]);
                        pa1[c >> 1] = ptx::pack_bf16(a1[0], a1[1]);
                    }
                    ptx::tmem_st8(sbase + 16 * u, pa0);
                    ptx::tmem_st8(sbase + BC + 16 * u, pa1);
                }
                ptx::tmem_wait_st();
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive(bar(C::B_PREADY + b));
                if (C::TRANSPOSED) ptx::mbar_arrive(bar(C::B_STEMPTY + j % TC_STATS_STAGES));
            }
            if (ok) ok = ptx::mbar_wait(bar(C::B_FINAL), 0, abort_flag, TC_WAIT_LIMIT_NS);
            if (ok) {
                ptx::tc_fence_after_sync();
                __nv_bfloat16* p0 = reinterpret_cast<__nv_bfloat16*>(p.out0) + ((size_t)bh * p.N + row0 + row) * p.d;
                __nv_bfloat16* p1 = reinterpret_cast<__nv_bfloat16*>(p.out1) + ((size_t)bh * p.N + row0 + row) * p.d;
                for (int ch = g; ch < ksteps; ch += 2) {
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
                    if (row_valid) {
                        *reinterpret_cast<uint4*>(p0 + 16 * ch) = make_uint4(q0[0], q0[1], q0[2], q0[3]);
                        *reinterpret_cast<uint4*>(p1 + 16 * ch) = make_uint4(q1[0], q1[1], q1[2], q1[3]);
                        if (16 * ch + 8 < p.d) {
                            *reinterpret_cast<uint4*>(p0 + 16 * ch + 8) = make_uint4(q0[4], q0[5], q0[6], q0[7]);
                            *reinterpret_cast<uint4*>(p1 + 16 * ch + 8) = make_uint4(q1[4], q1[5], q1[6], q1[7]);
                        }
                    }
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, 1);
}

}  // namespace tvm_attn
