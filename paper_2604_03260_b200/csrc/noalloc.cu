// focus_count_kept_noalloc: the exact attended-pair count for callers that cannot allocate device
// memory.  The only scratch the count needs -- the per-group column bitmaps of the key tiles --
// lives in a fixed array inside the library image instead of a caller-provided workspace.
#include "common.cuh"

#include <mutex>

namespace focus {

// Scratch: [batch*Hkv][nkt][K][4] uint32 words, at most FOCUS_NOALLOC_MAX_BYTES.  Every device that
// loads the library holds this array until the process exits.  In host code the name below is only
// a stand-in for the symbol; the device address is obtained with cudaGetSymbolAddress.
static __device__ __align__(256) uint32_t g_noalloc_gbits[FOCUS_NOALLOC_MAX_BYTES / 4];

constexpr int MAX_DEVICES = 64;
static uint32_t* g_scratch_addr[MAX_DEVICES];
static std::mutex g_scratch_mutex;

// Device address of the scratch array on the current device; looked up once per device and kept for
// the life of the process.  An application that destroys the device's primary context
// (cudaDeviceReset) invalidates the address: this entry point must not be used after that.
static int scratch_address(uint32_t** out) {
    int dev = 0;
    int rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
    if (rc) return rc;
    if (dev < 0 || dev >= MAX_DEVICES) return fail(FOCUS_ERR_UNSUPPORTED, "device ordinal %d is beyond %d", dev, MAX_DEVICES);
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        rc = check_cuda(cudaGetSymbolAddress(&p, g_noalloc_gbits), "cudaGetSymbolAddress(scratch)");
        if (rc) return rc;
        g_scratch_addr[dev] = static_cast<uint32_t*>(p);
    }
    *out = g_scratch_addr[dev];
    return FOCUS_OK;
}

// block of 128 threads per (key tile, KV head): word q of group g = ballot of "key 128 b + 32 q + lane is in g"
__global__ void __launch_bounds__(128)
noalloc_gbits_kernel(const uint32_t* __restrict__ mk, int n, int nkt, int K, uint32_t* __restrict__ gbits) {
    const int tile = blockIdx.x, head = blockIdx.y;
    const int tok = tile * 128 + threadIdx.x;
    const uint32_t v = tok < n ? mk[(size_t)head * n + tok] : 0u;
    uint32_t* gb = gbits + ((size_t)head * nkt + tile) * K * 4;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int g = 0; g < K; ++g) {
        const uint32_t word = __ballot_sync(0xffffffffu, (v >> g) & 1u);
        if (lane == 0) gb[g * 4 + warp] = word;
    }
}

// thread = query row; local keys counted in closed form, far keys by popcount over the bitmaps
__global__ void __launch_bounds__(128)
noalloc_count_kernel(const uint32_t* __restrict__ mq, const uint32_t* __restrict__ gbits, int G_heads, int Hq, int Hkv,
                     int n, int w, int K, int nkt, unsigned long long* __restrict__ out) {
    const int a = blockIdx.x, hq = blockIdx.y;
    const int hk = (hq / Hq) * Hkv + (hq % Hq) / G_heads;
    const int i = a * 128 + threadIdx.x;
    unsigned long long cnt = 0;
    if (i < n) {
        const uint32_t mi = mq[(size_t)hq * n + i];
        cnt = (unsigned long long)min(i, w) + 1ull;
        const long long nfar = (long long)i - w;
        for (long long k0 = 0; k0 < nfar; k0 += 128) {
            const uint32_t* gb = gbits + ((size_t)hk * nkt + (int)(k0 / 128)) * K * 4;
            uint32_t wd[4] = {0, 0, 0, 0};
            for (uint32_t rem = mi; rem; rem &= rem - 1) {
                const int g = __ffs(rem) - 1;
                if (g < K) {
                    const uint4 t = *reinterpret_cast<const uint4*>(gb + g * 4);
                    wd[0] |= t.x; wd[1] |= t.y; wd[2] |= t.z; wd[3] |= t.w;
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const long long lim = nfar - (k0 + q * 32);
                const uint32_t valid = lim >= 32 ? 0xffffffffu : (lim <= 0 ? 0u : ((1u << (int)lim) - 1u));
                cnt += __popc(wd[q] & valid);
            }
        }
    }
    for (int off = 16; off >= 1; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
    __shared__ unsigned long long s[4];
    if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = cnt;
    __syncthreads();
    if (threadIdx.x == 0) atomicAdd(&out[hq], s[0] + s[1] + s[2] + s[3]);
}

}  // namespace focus

extern "C" int focus_count_kept_noalloc(const focus_shape* shape, const uint32_t* mq, const uint32_t* mk,
                                        unsigned long long* counts_out, void* stream) {
    using namespace focus;
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (!mq || !mk || !counts_out) return fail(FOCUS_ERR_INVALID_ARG, "mq, mk or counts_out is NULL");
    const int HQ = shape->batch * shape->Hq, HK = shape->batch * shape->Hkv;
    const int nkt = cdiv(shape->n, 128), nqt = cdiv(shape->n, 128);
    const size_t need = (size_t)HK * nkt * shape->K * 16;
    if (need > (size_t)FOCUS_NOALLOC_MAX_BYTES)
        return fail(FOCUS_ERR_CAPACITY,
                    "focus_count_kept_noalloc needs %zu bytes of scratch (batch*Hkv*ceil(n/128)*K*16) but the built-in "
                    "array holds %d; use focus_count_kept with a caller-allocated workspace", need,
                    (int)FOCUS_NOALLOC_MAX_BYTES);
    // heads are the second grid dimension of both kernels: refuse before anything is enqueued
    if (HQ > 65535 || HK > 65535)
        return fail(FOCUS_ERR_UNSUPPORTED, "focus_count_kept_noalloc: batch*Hq (%d) and batch*Hkv (%d) must not exceed 65535", HQ, HK);
    if ((rc = require_sm100())) return rc;
    uint32_t* scratch = nullptr;
    if ((rc = scratch_address(&scratch))) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // counts start at zero; the bitmaps of the range in use are fully rewritten, nothing else is read
    if ((rc = check_cuda(cudaMemsetAsync(counts_out, 0, (size_t)HQ * sizeof(unsigned long long), st),
                         "cudaMemsetAsync(counts)")))
        return rc;
    noalloc_gbits_kernel<<<dim3(nkt, HK), 128, 0, st>>>(mk, shape->n, nkt, shape->K, scratch);
    noalloc_count_kernel<<<dim3(nqt, HQ), 128, 0, st>>>(mq, scratch, shape->Hq / shape->Hkv, shape->Hq, shape->Hkv,
                                                        shape->n, shape->window, shape->K, nkt, counts_out);
    return check_cuda(cudaGetLastError(), "focus_count_kept_noalloc kernels");
}
