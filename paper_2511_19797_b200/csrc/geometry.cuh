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

}  // namespace tvm_attn
