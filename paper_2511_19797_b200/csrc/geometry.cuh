// Where the rows of one side of an attention problem live in memory.  The query-side tensors (Q, tQ, O, tO, dO,
// dtO, dQ, dtQ) have M rows per head, the key-side tensors (K, V, tK, tV and their gradients) N rows (App. C
// "Background": Q in R^{M x d}, K, V in R^{N x d}); each side has its own element strides, so that a packed
// (B, H, rows, d) tensor and a (B, rows, H, d) slice of a fused projection are read in place alike.  The d
// elements of a row are always contiguous.
#pragma once
#include <stddef.h>

namespace tvm_attn {

struct Geom {
    int rows;               // rows per head
    long long rs, hs, bs;   // element stride between rows, heads, batches
    // element offset of row 0 of flat head index bh = b * H + h
    __host__ __device__ __forceinline__ size_t head_off(int bh, int H) const {
        const int b = bh / H, h = bh - b * H;
        return (size_t)b * (size_t)bs + (size_t)h * (size_t)hs;
    }
};

#ifdef __CUDACC__
// Sum of v over the `gs` consecutive lanes of a warp that share a row (lanes sub * gs .. sub * gs + gs - 1), returned
// to all of them.  A power-of-two group is a butterfly; any other size (nine 16-byte chunks for d = 72) has its first
// lane collect the others' values and broadcast the total, which keeps 27 of 32 lanes busy where rounding the group
// up to 16 lanes would leave 14 idle.  Executed by the whole warp.
__device__ __forceinline__ float lane_group_sum(float v, int gs, int lane) {
    if ((gs & (gs - 1)) == 0) {
        for (int off = gs >> 1; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        return v;
    }
    float acc = v;
    for (int k = 1; k < gs; ++k) acc += __shfl_sync(0xffffffffu, v, lane + k);   // right on the group's first lane
    return __shfl_sync(0xffffffffu, acc, lane - lane % gs);
}

// Rows of 2 d bytes, lane = row, 32 bytes (lo, hi) of its row per lane: written 16 bytes per lane, one warp
// instruction touches 32 half sectors in 32 cache lines.  This helper pairs the lanes instead: lanes 2 i and
// 2 i + 1 write the two halves of ONE row's 32 bytes, the even row in a first instruction and the odd row in a
// second, and swap a half between them, so that each instruction writes 16 complete 32-byte sectors in 16 lines.
// (The same pairing for the loads of the owner rows measured slower.)
// `chunk`: this lane's 32 bytes in its own row; `pitch`: elements between rows; ok_even / ok_odd: the pair's rows
// exist; has_hi: the upper 16 bytes exist (d is a multiple of 8, not of 16).  Executed by the whole warp.
template <typename T>
__device__ __forceinline__ void store_row_pairs(T* chunk, long long pitch, int lane, bool ok_even, bool ok_odd, bool has_hi,
                                                const uint4& lo, const uint4& hi) {
    const bool odd = lane & 1;
    const uint4 x = odd ? lo : hi;   // the even lane hands over its upper half, the odd lane its lower one
    uint4 y;
    y.x = __shfl_xor_sync(0xffffffffu, x.x, 1);
    y.y = __shfl_xor_sync(0xffffffffu, x.y, 1);
    y.z = __shfl_xor_sync(0xffffffffu, x.z, 1);
    y.w = __shfl_xor_sync(0xffffffffu, x.w, 1);
    T* even_row = odd ? chunk - pitch : chunk;
    T* odd_row = odd ? chunk : chunk + pitch;
    const int half = odd ? 16 / (int)sizeof(T) : 0;
    if (ok_even && (!odd || has_hi)) *reinterpret_cast<uint4*>(even_row + half) = odd ? y : lo;
    if (ok_odd && (!odd || has_hi)) *reinterpret_cast<uint4*>(odd_row + half) = odd ? hi : y;
}
#endif

}  // namespace tvm_attn
