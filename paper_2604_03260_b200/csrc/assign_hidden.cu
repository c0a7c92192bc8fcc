// focus_assign_hidden: the router as the paper states it (Sec. 2 "Learned grouping", Eq. 1): one
// routing vector per token, W_g h_i in d_g dimensions, scored against the centroids by dot product;
// the token joins its top-k groups and every head (query and key role alike) uses that mask.
//
// W_g^T h . C_g = h . (W_g C_g), so the projection and the centroids fold into K vectors of length d
// (a small kernel, once per call); scoring then reads each hidden state exactly once, which makes the
// pass HBM-bound: 2 d bytes per token.  Thread = token; the block's rows stream through shared
// memory in chunks of 64 elements (coalesced asynchronous 16-byte copies, two chunks in flight).
#include "common.cuh"

namespace focus {

constexpr int AH_THREADS = 64;       // tokens per block (small, so that modest sequence lengths still fill the GPU)
constexpr int AH_CHUNK = 64;         // elements of a row per stage
constexpr int AH_ROWB = 2 * AH_CHUNK + 16;   // padded row: conflict-free 16-byte reads per token

// folded[g][e] = sum_j Wg[e][j] * C[g][j]
__global__ void __launch_bounds__(256)
fold_router_kernel(const float* __restrict__ Wg, const float* __restrict__ C, int d, int dg, int K, float* __restrict__ folded) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    const int g = blockIdx.y;
    if (e >= d) return;
    float s = 0.f;
    for (int j = 0; j < dg; ++j) s = fmaf(Wg[(size_t)e * dg + j], C[(size_t)g * dg + j], s);
    folded[(size_t)g * d + e] = s;
}

template <int KMAX>
__global__ void __launch_bounds__(AH_THREADS)
assign_hidden_kernel(const __nv_bfloat16* __restrict__ h, int64_t stride_b, int64_t stride_n, int n, int d, int K, int topk,
                     const float* __restrict__ folded, const float* __restrict__ bias, int Hq, int Hkv,
                     uint32_t* __restrict__ mq, uint32_t* __restrict__ mk, unsigned long long* near_ties, float eps,
                     float* __restrict__ scores) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned char* tile = smem_raw;                                           // [2][AH_THREADS][AH_ROWB]
    float* cs = reinterpret_cast<float*>(smem_raw + 2 * AH_THREADS * AH_ROWB);   // [2][KMAX][AH_CHUNK]
    const int b = blockIdx.y;
    const int tok0 = blockIdx.x * AH_THREADS;
    const int tok = tok0 + threadIdx.x;
    const bool in = tok < n;
    const __nv_bfloat16* hb = h + (size_t)b * stride_b;
    const int nchunk = (d + AH_CHUNK - 1) / AH_CHUNK;

    auto stage = [&](int ch, int buf) {
        const int e0 = ch * AH_CHUNK;
        const int vec = min(AH_CHUNK, d - e0) / 8;                            // 16-byte pieces per row in this chunk
        for (int q = threadIdx.x; q < AH_THREADS * vec; q += AH_THREADS) {
            const int r = q / vec, c = q % vec;
            if (tok0 + r < n) {
                const uint32_t dst = (uint32_t)__cvta_generic_to_shared(tile + ((size_t)buf * AH_THREADS + r) * AH_ROWB + c * 16);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(hb + (size_t)(tok0 + r) * stride_n + e0 + c * 8)
                             : "memory");
            }
        }
        for (int q = threadIdx.x; q < KMAX * (AH_CHUNK / 4); q += AH_THREADS) {   // folded centroids of the chunk, 16 bytes each
            const int g = q / (AH_CHUNK / 4), c = q % (AH_CHUNK / 4);
            float* dstp = cs + ((size_t)buf * KMAX + g) * AH_CHUNK + c * 4;
            if (g < K && e0 + c * 4 < d) {
                const uint32_t dst = (uint32_t)__cvta_generic_to_shared(dstp);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(folded + (size_t)g * d + e0 + c * 4) : "memory");
            } else {
                *reinterpret_cast<float4*>(dstp) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    float2 dot2[KMAX];
#pragma unroll
    for (int g = 0; g < KMAX; ++g) dot2[g] = make_float2(0.f, 0.f);
    stage(0, 0);
    for (int ch = 0; ch < nchunk; ++ch) {
        const int buf = ch & 1;
        if (ch + 1 < nchunk) {
            stage(ch + 1, buf ^ 1);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();
        const int vec = min(AH_CHUNK, d - ch * AH_CHUNK) / 8;
        const unsigned char* row = tile + ((size_t)buf * AH_THREADS + threadIdx.x) * AH_ROWB;
        const float* cb = cs + (size_t)buf * KMAX * AH_CHUNK;
#pragma unroll 4
        for (int v = 0; v < vec; ++v) {
            const uint4 rv = in ? *reinterpret_cast<const uint4*>(row + v * 16) : make_uint4(0, 0, 0, 0);
            const uint32_t wds[4] = {rv.x, rv.y, rv.z, rv.w};
            float2 xv[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) xv[e] = make_float2(__uint_as_float(wds[e] << 16), __uint_as_float(wds[e] & 0xffff0000u));
#pragma unroll
            for (int g = 0; g < KMAX; ++g) {
                const float4 c0 = *reinterpret_cast<const float4*>(cb + g * AH_CHUNK + v * 8);
                const float4 c1 = *reinterpret_cast<const float4*>(cb + g * AH_CHUNK + v * 8 + 4);
                float2 sacc = dot2[g];
                sacc = __ffma2_rn(xv[0], make_float2(c0.x, c0.y), sacc);
                sacc = __ffma2_rn(xv[1], make_float2(c0.z, c0.w), sacc);
                sacc = __ffma2_rn(xv[2], make_float2(c1.x, c1.y), sacc);
                sacc = __ffma2_rn(xv[3], make_float2(c1.z, c1.w), sacc);
                dot2[g] = sacc;
            }
        }
        __syncthreads();            // the buffer is refilled two iterations later
    }
    float score[KMAX];
#pragma unroll
    for (int g = 0; g < KMAX; ++g) score[g] = dot2[g].x + dot2[g].y + ((bias && g < K) ? __ldg(bias + g) : 0.f);
    if (scores) {   // the scores themselves (training-time soft assignment), rows of KMAX floats, zero beyond K
        if (in) {
            float4* o = reinterpret_cast<float4*>(scores + ((size_t)b * n + tok) * KMAX);
#pragma unroll
            for (int c = 0; c < KMAX / 4; ++c)
                o[c] = make_float4(4 * c < K ? score[4 * c] : 0.f, 4 * c + 1 < K ? score[4 * c + 1] : 0.f,
                                   4 * c + 2 < K ? score[4 * c + 2] : 0.f, 4 * c + 3 < K ? score[4 * c + 3] : 0.f);
        }
        return;
    }
    uint32_t taken = 0;
    float last = 0.f, next = 0.f;
    // topk picks, then one more to measure the margin; strict '>' keeps the lowest index on ties
    for (int it = 0; it <= topk && it < K; ++it) {
        float best = -INFINITY;
        int bi = 0;
#pragma unroll
        for (int g = 0; g < KMAX; ++g) {
            const bool ok = g < K && !((taken >> g) & 1u) && (score[g] > best || best == -INFINITY);
            if (ok) { best = score[g]; bi = g; }
        }
        if (it < topk) { taken |= 1u << bi; last = best; }
        else next = best;
    }
    if (in) {   // every head of the layer shares the token's mask
        if (mq) for (int hh = 0; hh < Hq; ++hh) mq[((size_t)b * Hq + hh) * n + tok] = taken;
        if (mk) for (int hh = 0; hh < Hkv; ++hh) mk[((size_t)b * Hkv + hh) * n + tok] = taken;
    }
    if (near_ties) {
        const unsigned int near = __ballot_sync(0xffffffffu, in && topk < K && (last - next) < eps);
        if ((threadIdx.x & 31) == 0 && near) atomicAdd(near_ties, (unsigned long long)__popc(near));
    }
}

template <int KMAX>
static int launch_k(const focus_shape* s, const void* h, int64_t sb, int64_t sn, int d, const float* folded, const float* bias,
                    uint32_t* mq, uint32_t* mk, unsigned long long* near_ties, float eps, float* scores, cudaStream_t st) {
    const size_t smem = (size_t)2 * AH_THREADS * AH_ROWB + (size_t)2 * KMAX * AH_CHUNK * sizeof(float);
    auto kern = assign_hidden_kernel<KMAX>;
    int rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem),
                        "cudaFuncSetAttribute(assign_hidden)");
    if (rc) return rc;
    kern<<<dim3(cdiv(s->n, AH_THREADS), s->batch), AH_THREADS, smem, st>>>(
        reinterpret_cast<const __nv_bfloat16*>(h), sb, sn, s->n, d, s->K, s->topk, folded, bias, s->Hq, s->Hkv, mq, mk, near_ties, eps,
        scores);
    return check_cuda(cudaGetLastError(), "assign_hidden kernel launch");
}

int launch_assign_hidden(const focus_shape* s, const void* h, int64_t sb, int64_t sn, int d, int dg, const float* Wg,
                         const float* C, const float* bias, float* folded, uint32_t* mq, uint32_t* mk,
                         unsigned long long* near_ties, float eps, float* scores, cudaStream_t st) {
    fold_router_kernel<<<dim3(cdiv(d, 256), s->K), 256, 0, st>>>(Wg, C, d, dg, s->K, folded);
    int rc = check_cuda(cudaGetLastError(), "fold_router kernel launch");
    if (rc) return rc;
    if (s->K <= 4) return launch_k<4>(s, h, sb, sn, d, folded, bias, mq, mk, near_ties, eps, scores, st);
    if (s->K <= 8) return launch_k<8>(s, h, sb, sn, d, folded, bias, mq, mk, near_ties, eps, scores, st);
    if (s->K <= 16) return launch_k<16>(s, h, sb, sn, d, folded, bias, mq, mk, near_ties, eps, scores, st);
    return launch_k<32>(s, h, sb, sn, d, folded, bias, mq, mk, near_ties, eps, scores, st);
}

}  // namespace focus
