// focus_assign: cosine of every head vector with the K centroids of its KV head, top-k membership
// mask out (paper Eq. 1 + the top-k rule of Sec. 3.6).  HBM-bound: each vector is read once with
// 16-byte loads; the centroids of the block's KV head sit in shared memory.
#include "common.cuh"

namespace focus {

constexpr int ASSIGN_THREADS = 256;
constexpr int ASSIGN_TOKENS = 512;   // tokens of one head per block

template <int D, int KMAX>
__global__ void __launch_bounds__(ASSIGN_THREADS)
assign_kernel(const __nv_bfloat16* __restrict__ x, int64_t stride_b, int64_t stride_h, int64_t stride_n,
              int H, int G, int n, int K, int topk, const float* __restrict__ C,
              uint32_t* __restrict__ masks, unsigned long long* near_ties, float eps) {
    constexpr int LPV = D / 8;            // lanes per vector (16 bytes each)
    constexpr int VPW = 32 / LPV;         // vectors per warp per step
    constexpr int VEC = KMAX <= 8 ? 4 : (KMAX == 16 ? 2 : 1);   // vectors in flight per lane
    constexpr int WARPS = ASSIGN_THREADS / 32;
    constexpr int PER_ROUND = WARPS * VPW * VEC;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* cs = reinterpret_cast<float*>(smem_raw);            // [K][D]
    float* cinv = cs + KMAX * D;                               // [KMAX] 1/|c_g|
    uint32_t* mstage = reinterpret_cast<uint32_t*>(cinv + KMAX);   // [ASSIGN_TOKENS]
    __shared__ unsigned int s_near;

    const int bh = blockIdx.y;
    const int b = bh / H, h = bh % H;
    const int hk = h / G;
    const int tok0 = blockIdx.x * ASSIGN_TOKENS;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    for (int i = threadIdx.x; i < K * D; i += ASSIGN_THREADS) cs[i] = C[(size_t)hk * K * D + i];
    if (threadIdx.x == 0) s_near = 0;
    __syncthreads();
    if (warp < 1) {
        for (int g = lane; g < KMAX; g += 32) {
            float s = 0.f;
            if (g < K)
                for (int d = 0; d < D; ++d) s = fmaf(cs[g * D + d], cs[g * D + d], s);
            cinv[g] = s > 0.f ? rsqrtf(s) : 0.f;
        }
    }
    __syncthreads();

    const __nv_bfloat16* xb = x + (size_t)b * stride_b + (size_t)h * stride_h;
    const int sub = lane / LPV;           // which vector of the warp's VPW
    const int part = lane % LPV;          // which 8-element slice
    unsigned int near_local = 0;

    for (int round = 0; round < ASSIGN_TOKENS / PER_ROUND; ++round) {
        float xv[VEC][8];
        int tloc[VEC];
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
            tloc[v] = round * PER_ROUND + (v * WARPS + warp) * VPW + sub;
            const int tok = tok0 + tloc[v];
            uint4 raw = make_uint4(0, 0, 0, 0);
            if (tok < n) raw = *reinterpret_cast<const uint4*>(xb + (size_t)tok * stride_n + part * 8);
            const uint32_t wds[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                xv[v][2 * e] = __uint_as_float(wds[e] << 16);
                xv[v][2 * e + 1] = __uint_as_float(wds[e] & 0xffff0000u);
            }
        }
        float dot[VEC][KMAX];
        float xx[VEC];
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
            xx[v] = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) xx[v] = fmaf(xv[v][e], xv[v][e], xx[v]);
        }
#pragma unroll
        for (int g = 0; g < KMAX; ++g) {
            float c[8];
            if (g < K) {
                const float4 c0 = *reinterpret_cast<const float4*>(cs + g * D + part * 8);
                const float4 c1 = *reinterpret_cast<const float4*>(cs + g * D + part * 8 + 4);
                c[0] = c0.x; c[1] = c0.y; c[2] = c0.z; c[3] = c0.w;
                c[4] = c1.x; c[5] = c1.y; c[6] = c1.z; c[7] = c1.w;
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) c[e] = 0.f;
            }
#pragma unroll
            for (int v = 0; v < VEC; ++v) {
                float s = 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) s = fmaf(xv[v][e], c[e], s);
                dot[v][g] = s;
            }
        }
        // sum the slices of each vector (butterfly inside groups of LPV lanes)
#pragma unroll
        for (int off = LPV / 2; off >= 1; off >>= 1) {
#pragma unroll
            for (int v = 0; v < VEC; ++v) {
                xx[v] += __shfl_xor_sync(0xffffffffu, xx[v], off);
#pragma unroll
                for (int g = 0; g < KMAX; ++g) dot[v][g] += __shfl_xor_sync(0xffffffffu, dot[v][g], off);
            }
        }
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
            const float xinv = xx[v] > 0.f ? rsqrtf(xx[v]) : 0.f;
            float cosv[KMAX];
#pragma unroll
            for (int g = 0; g < KMAX; ++g) cosv[g] = dot[v][g] * cinv[g] * xinv;
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
            if (part == 0) {
                mstage[tloc[v]] = taken;
                if (topk < K && tok0 + tloc[v] < n && (last - next) < eps) ++near_local;
            }
        }
    }
    if (near_local) atomicAdd(&s_near, near_local);
    __syncthreads();
    uint32_t* mo = masks + (size_t)bh * n;
    for (int i = threadIdx.x; i < ASSIGN_TOKENS; i += ASSIGN_THREADS)
        if (tok0 + i < n) mo[tok0 + i] = mstage[i];
    if (threadIdx.x == 0 && near_ties && s_near) atomicAdd(near_ties, (unsigned long long)s_near);
}

template <int D, int KMAX>
static int launch_one(const focus_shape* s, const focus_tensor& x, int H, const float* C, uint32_t* masks,
                      unsigned long long* near_ties, float eps, cudaStream_t st) {
    const size_t smem = (size_t)(KMAX * D + KMAX) * sizeof(float) + ASSIGN_TOKENS * sizeof(uint32_t);
    auto kern = assign_kernel<D, KMAX>;
    int rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem),
                        "cudaFuncSetAttribute(assign)");
    if (rc) return rc;
    dim3 grid(cdiv(s->n, ASSIGN_TOKENS), s->batch * H);
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
