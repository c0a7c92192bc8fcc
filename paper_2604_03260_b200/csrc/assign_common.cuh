// Pieces shared by the two group-assignment kernels (head vectors against per-head centroids; hidden states
// against the folded router): the swizzled operand layout, the three-term bf16 split, the top-k selection.
#pragma once
#include "common.cuh"

namespace focus {

// byte offset of element (row, col) inside a K-major tile of `rows` rows stored as 64-column sub-tiles with the
// 128-byte swizzle the MMA descriptors use (16-byte chunk index XOR row mod 8)
__device__ __forceinline__ uint32_t sw128_offset(int row, int col, int rows) {
    const int sub = col >> 6, c = col & 63;
    return (uint32_t)(sub * rows * 128 + row * 128 + ((((c * 2) >> 4) ^ (row & 7)) << 4) + ((c * 2) & 15));
}

// v = hi + mid + lo with bf16 terms: 24 mantissa bits, so a product of v with a bf16 number is the sum of three
// exact bf16 x bf16 products
__device__ __forceinline__ void split3_bf16(float v, __nv_bfloat16& hi, __nv_bfloat16& mid, __nv_bfloat16& lo) {
    hi = __float2bfloat16_rn(v);
    v -= __bfloat162float(hi);
    mid = __float2bfloat16_rn(v);
    v -= __bfloat162float(mid);
    lo = __float2bfloat16_rn(v);
}

// The `topk` best of val[0..K) as a bit mask (paper Sec. 3.6: top-k membership), an exact tie going to the lower
// index; `last` is the worst value taken and `next` the best one left (their difference is the margin a near-tie
// is judged by; `next` is meaningless when topk >= K).  val[g] for g >= K is overwritten.
template <int KMAX>
__device__ __forceinline__ uint32_t select_topk(float (&val)[KMAX], int K, int topk, float& last, float& next) {
    uint32_t taken = 0;
    last = 0.f;
    next = 0.f;
    if constexpr (KMAX <= 8) {
        // rank of every group among the K (how many beat it): rank < topk is taken
        int rank[KMAX];
#pragma unroll
        for (int g = 0; g < KMAX; ++g) {
            rank[g] = 0;
            if (g >= K) val[g] = -INFINITY;
        }
#pragma unroll
        for (int a = 0; a < KMAX; ++a)
#pragma unroll
            for (int c = a + 1; c < KMAX; ++c) {
                const bool a_first = !(val[c] > val[a]);
                rank[c] += a_first ? 1 : 0;
                rank[a] += a_first ? 0 : 1;
            }
        const int kk = topk < K ? topk : K;
#pragma unroll
        for (int g = 0; g < KMAX; ++g) {
            if (g < K && rank[g] < kk) taken |= 1u << g;
            if (rank[g] == kk - 1) last = val[g];
            if (rank[g] == kk) next = val[g];
        }
    } else {
        // topk picks, then one more to measure the margin; strict '>' keeps the lowest index on ties
        for (int it = 0; it <= topk && it < K; ++it) {
            float best = -INFINITY;
            int bi = 0;
#pragma unroll
            for (int g = 0; g < KMAX; ++g) {
                const bool better = g < K && !((taken >> g) & 1u) && (val[g] > best || best == -INFINITY);
                if (better) { best = val[g]; bi = g; }
            }
            if (it < topk) { taken |= 1u << bi; last = best; }
            else next = best;
        }
    }
    return taken;
}

}  // namespace focus
