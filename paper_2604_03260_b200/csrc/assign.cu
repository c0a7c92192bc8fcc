// focus_assign: cosine of every head vector with the K centroids of its KV head, top-k membership
// mask out (paper Eq. 1 + the top-k rule of Sec. 3.6).  HBM-bound: each vector is read once with
// 16-byte loads by the one thread that owns the token; the centroids of the block's KV head sit in
// shared memory.
#include "common.cuh"

namespace focus {

constexpr int ASSIGN_THREADS = 128;   // one thread per token: 128 tokens of one head per block

// Thread = token.  The block copies its 128 rows into shared memory with coalesced asynchronous 16-byte
// copies (all in flight at once); each thread then reads its own row, accumulates |x|^2 and the K dot products
// against the centroids held in shared memory (every lane reads the same centroid words: broadcast,
// no bank conflicts), then selects its top-k groups and writes its mask word (coalesced).
template <int D, int KMAX>
__global__ void __launch_bounds__(ASSIGN_THREADS)
assign_kernel(const __nv_bfloat16* __restrict__ x, int64_t stride_b, int64_t stride_h, int64_t stride_n,
              int H, int G, int n, int K, int topk, const float* __restrict__ C,
              uint32_t* __restrict__ masks, unsigned long long* near_ties, float eps) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* cs = reinterpret_cast<float*>(smem_raw);            // [KMAX][D], rows >= K are zero
    float* cinv = cs + KMAX * D;                               // [KMAX] 1/|c_g|
    unsigned char* tile = reinterpret_cast<unsigned char*>(cinv + KMAX);   // [ASSIGN_THREADS] rows of 2D + 16 bytes
    constexpr int ROWB = 2 * D + 16;                           // padded row: conflict-free 16-byte reads per token

    const int bh = blockIdx.y;
    const int b = bh / H, h = bh % H;
    const int hk = h / G;
    const int tok = blockIdx.x * ASSIGN_THREADS + threadIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool in = tok < n;

    // the block's rows first, as coalesced asynchronous 16-byte copies into shared memory (consecutive
    // threads copy consecutive chunks of a row); they overlap the staging of the centroids
    {
        const __nv_bfloat16* xh = x + (size_t)b * stride_b + (size_t)h * stride_h;
        const int tok0 = blockIdx.x * ASSIGN_THREADS;
#pragma unroll
        for (int i = 0; i < D / 8; ++i) {
            const int q = i * ASSIGN_THREADS + threadIdx.x;
            const int r = q / (D / 8), c = q % (D / 8);
            if (tok0 + r < n) {
                const uint32_t dst = (uint32_t)__cvta_generic_to_shared(tile + r * ROWB + c * 16);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(xh + (size_t)(tok0 + r) * stride_n + c * 8)
                             : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    }

    for (int i = threadIdx.x; i < KMAX * D; i += ASSIGN_THREADS) cs[i] = i < K * D ? C[(size_t)hk * K * D + i] : 0.f;
    __syncthreads();
    for (int g = warp; g < KMAX; g += ASSIGN_THREADS / 32) {      // one warp per centroid norm
        float s = 0.f;
        for (int d = lane; d < D; d += 32) s = fmaf(cs[g * D + d], cs[g * D + d], s);
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (lane == 0) cinv[g] = s > 0.f ? rsqrtf(s) : 0.f;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();

    // packed fp32 pairs: even elements accumulate in .x, odd elements in .y
    float2 xx2 = make_float2(0.f, 0.f);
    float2 dot2[KMAX];
#pragma unroll
    for (int g = 0; g < KMAX; ++g) dot2[g] = make_float2(0.f, 0.f);
#pragma unroll
    for (int v = 0; v < D / 8; ++v) {
        const uint4 rv = in ? *reinterpret_cast<const uint4*>(tile + threadIdx.x * ROWB + v * 16) : make_uint4(0, 0, 0, 0);
        const uint32_t wds[4] = {rv.x, rv.y, rv.z, rv.w};
        float2 xv[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) xv[e] = make_float2(__uint_as_float(wds[e] << 16), __uint_as_float(wds[e] & 0xffff0000u));
#pragma unroll
        for (int e = 0; e < 4; ++e) xx2 = __ffma2_rn(xv[e], xv[e], xx2);
#pragma unroll
        for (int g = 0; g < KMAX; ++g) {
            const float4 c0 = *reinterpret_cast<const float4*>(cs + g * D + v * 8);
            const float4 c1 = *reinterpret_cast<const float4*>(cs + g * D + v * 8 + 4);
            float2 sacc = dot2[g];
            sacc = __ffma2_rn(xv[0], make_float2(c0.x, c0.y), sacc);
            sacc = __ffma2_rn(xv[1], make_float2(c0.z, c0.w), sacc);
            sacc = __ffma2_rn(xv[2], make_float2(c1.x, c1.y), sacc);
            sacc = __ffma2_rn(xv[3], make_float2(c1.z, c1.w), sacc);
            dot2[g] = sacc;
        }
    }
    const float xx = xx2.x + xx2.y;
    float dot[KMAX];
#pragma unroll
    for (int g = 0; g < KMAX; ++g) dot[g] = dot2[g].x + dot2[g].y;
    const float xinv = xx > 0.f ? rsqrtf(xx) : 0.f;
    float cosv[KMAX];
#pragma unroll
    for (int g = 0; g < KMAX; ++g) cosv[g] = dot[g] * cinv[g] * xinv;
    uint32_t taken = 0;
    float last = 0.f, next = 0.f;
    // topk picks, then one more to measure the margin; strict '>' keeps the lowest index on ties
    for (int it = 0; it <= topk && it < K; ++it) {
        float best = -INFINITY;
        int bi = 0;
#pragma unroll
        for (int g = 0; g < KMAX; ++g) {
            const bool ok = g < K && !((taken >> g) & 1u) && (cosv[g] > best || best == -INFINITY);
            if (ok) { best = cosv[g]; bi = g; }
        }
        if (it < topk) { taken |= 1u << bi; last = best; }
        else next = best;
    }
    if (in) masks[(size_t)bh * n + tok] = taken;
    if (near_ties) {
        const unsigned int near = __ballot_sync(0xffffffffu, in && topk < K && (last - next) < eps);
        if (lane == 0 && near) atomicAdd(near_ties, (unsigned long long)__popc(near));
    }
}

template <int D, int KMAX>
static int launch_one(const focus_shape* s, const focus_tensor& x, int H, const float* C, uint32_t* masks,
                      unsigned long long* near_ties, float eps, cudaStream_t st) {
    const size_t smem = (size_t)(KMAX * D + KMAX) * sizeof(float) + (size_t)ASSIGN_THREADS * (2 * D + 16);
    auto kern = assign_kernel<D, KMAX>;
    int rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem),
                        "cudaFuncSetAttribute(assign)");
    if (rc) return rc;
    dim3 grid(cdiv(s->n, ASSIGN_THREADS), s->batch * H);
    kern<<<grid, ASSIGN_THREADS, smem, st>>>(reinterpret_cast<const __nv_bfloat16*>(x.ptr), x.stride_b, x.stride_h,
                                              x.stride_n, H, H / s->Hkv, s->n, s->K, s->topk, C, masks, near_ties, eps);
    return check_cuda(cudaGetLastError(), "assign kernel launch");
}

template <int D>
static int launch_d(const focus_shape* s, const focus_tensor& x, int H, const float* C, uint32_t* masks,
                    unsigned long long* near_ties, float eps, cudaStream_t st) {
    if (s->K <= 4) return launch_one<D, 4>(s, x, H, C, masks, near_ties, eps, st);
    if (s->K <= 8) return launch_one<D, 8>(s, x, H, C, masks, near_ties, eps, st);
    if (s->K <= 16) return launch_one<D, 16>(s, x, H, C, masks, near_ties, eps, st);
    return launch_one<D, 32>(s, x, H, C, masks, near_ties, eps, st);
}

int launch_assign(const focus_shape* s, const focus_tensor& x, int H, const float* C, uint32_t* masks,
                  unsigned long long* near_ties, float eps, cudaStream_t st) {
    switch (s->D) {
        case 64: return launch_d<64>(s, x, H, C, masks, near_ties, eps, st);
        case 128: return launch_d<128>(s, x, H, C, masks, near_ties, eps, st);
        case 256: return launch_d<256>(s, x, H, C, masks, near_ties, eps, st);
    }
    return fail(FOCUS_ERR_UNSUPPORTED, "D (%d) must be 64, 128 or 256", s->D);
}

}  // namespace focus
