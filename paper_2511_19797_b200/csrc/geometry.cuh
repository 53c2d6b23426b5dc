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
#endif

}  // namespace tvm_attn
