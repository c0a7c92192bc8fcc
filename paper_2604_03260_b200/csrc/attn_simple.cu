// A deliberately plain attention kernel used for debugging the tensor-core path
// (FOCUS_ATTN_IMPL=simple): one warp per query row, the attended-pair rule evaluated pair by pair
// straight from the masks (no tile structures), fp32 online softmax on CUDA cores.
#include "common.cuh"

namespace focus {

template <int D>
__global__ void __launch_bounds__(256)
attn_simple_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                   const __nv_bfloat16* __restrict__ v, __nv_bfloat16* __restrict__ o, focus_tensor tq, focus_tensor tk,
                   focus_tensor tv, focus_tensor to, const uint32_t* __restrict__ mq, const uint32_t* __restrict__ mk,
                   int dense, int B, int Hq, int Hkv, int n, int w, float scale, float softcap, float* __restrict__ lse) {
    constexpr int E = D / 32;
    const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= (long long)B * Hq * n) return;
    const int i = (int)(row % n);
    const int hq = (int)(row / n);
    const int b = hq / Hq, h = hq % Hq;
    const int G = Hq / Hkv;
    const int hk = b * Hkv + h / G;
    const __nv_bfloat16* qp = q + (size_t)b * tq.stride_b + (size_t)h * tq.stride_h + (size_t)i * tq.stride_n;
    const __nv_bfloat16* kb = k + (size_t)b * tk.stride_b + (size_t)(h / G) * tk.stride_h;
    const __nv_bfloat16* vb = v + (size_t)b * tv.stride_b + (size_t)(h / G) * tv.stride_h;
    float qv[E], acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) { qv[e] = __bfloat162float(qp[lane * E + e]) * scale; acc[e] = 0.f; }
    const uint32_t mi = dense ? 0xffffffffu : mq[(size_t)hq * n + i];
    float m = -INFINITY, l = 0.f;
    for (int j0 = 0; j0 <= i; j0 += 32) {
        const int j = j0 + lane;
        bool keep = j <= i;
        if (keep && !dense) keep = (i - j <= w) || ((mi & mk[(size_t)hk * n + j]) != 0u);
        uint32_t bal = __ballot_sync(0xffffffffu, keep);
        while (bal) {
            const int jj = j0 + __ffs(bal) - 1;
            bal &= bal - 1;
            const __nv_bfloat16* kp = kb + (size_t)jj * tk.stride_n + lane * E;
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < E; ++e) s = fmaf(qv[e], __bfloat162float(kp[e]), s);
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
            if (softcap > 0.f) s = softcap * tanhf(s / softcap);
            const float mn = fmaxf(m, s);
            const float corr = __expf(m - mn);      // m = -inf on the first key: exp(-inf) = 0
            const float p = __expf(s - mn);
            l = l * corr + p;
            const __nv_bfloat16* vp = vb + (size_t)jj * tv.stride_n + lane * E;
#pragma unroll
            for (int e = 0; e < E; ++e) acc[e] = fmaf(p, __bfloat162float(vp[e]), acc[e] * corr);
            m = mn;
        }
    }
    __nv_bfloat16* op = o + (size_t)b * to.stride_b + (size_t)h * to.stride_h + (size_t)i * to.stride_n;
    const float inv = 1.f / l;
#pragma unroll
    for (int e = 0; e < E; ++e) op[lane * E + e] = __float2bfloat16(acc[e] * inv);
    if (lane == 0) lse[(size_t)hq * n + i] = m + logf(l);
}

template <int D>
static int launch_simple_d(const AttnArgs& a, cudaStream_t st) {
    const long long rows = (long long)a.s.batch * a.s.Hq * a.s.n;
    const long long blocks = (rows + 7) / 8;
    if (blocks > 0x7fffffffLL) return fail(FOCUS_ERR_UNSUPPORTED, "too many rows for the debug kernel");
    attn_simple_kernel<D><<<(unsigned)blocks, 256, 0, st>>>(
        (const __nv_bfloat16*)a.q.ptr, (const __nv_bfloat16*)a.k.ptr, (const __nv_bfloat16*)a.v.ptr,
        (__nv_bfloat16*)a.o.ptr, a.q, a.k, a.v, a.o, a.mq, a.mk, a.ws ? 0 : 1, a.s.batch, a.s.Hq, a.s.Hkv, a.s.n,
        a.s.window, a.scale, a.s.softcap, a.lse);
    return check_cuda(cudaGetLastError(), "attn_simple kernel");
}

int launch_attn_simple(const AttnArgs& a, cudaStream_t st) {
    switch (a.s.D) {
        case 64: return launch_simple_d<64>(a, st);
        case 128: return launch_simple_d<128>(a, st);
        case 256: return launch_simple_d<256>(a, st);
    }
    return fail(FOCUS_ERR_UNSUPPORTED, "D (%d) must be 64, 128 or 256", a.s.D);
}

}  // namespace focus
