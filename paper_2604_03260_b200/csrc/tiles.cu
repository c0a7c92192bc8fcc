// focus_build_tiles / focus_count_kept: integer-only passes over the membership masks.
//   summaries   OR/AND of the masks of each 128-token tile, per-group column bitmaps of key tiles
//   live set    far tile pairs whose OR summaries intersect (everything else far is skipped)
//   kept count  exact number of attended pairs per query head
#include "common.cuh"

namespace focus {

constexpr int TM = FOCUS_TILE_M;
constexpr int TN = FOCUS_TILE_N;

// One block of 128 threads per (head, tile).  side = 0: query masks, 1: key masks (+ gbits).
__global__ void __launch_bounds__(128)
summarise_kernel(const uint32_t* __restrict__ m, int n, int nt, int K, uint32_t* __restrict__ orv,
                 uint32_t* __restrict__ andv, uint32_t* __restrict__ gbits) {
    const int tile = blockIdx.x, head = blockIdx.y;
    const int tok = tile * 128 + threadIdx.x;
    const bool in = tok < n;
    const uint32_t v = in ? m[(size_t)head * n + tok] : 0u;
    uint32_t o = v, a = in ? v : 0xffffffffu;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        o |= __shfl_xor_sync(0xffffffffu, o, off);
        a &= __shfl_xor_sync(0xffffffffu, a, off);
    }
    __shared__ uint32_t so[4], sa[4];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { so[warp] = o; sa[warp] = a; }
    if (gbits) {
        uint32_t* gb = gbits + ((size_t)head * nt + tile) * K * 4;
        for (int g = 0; g < K; ++g) {
            const uint32_t word = __ballot_sync(0xffffffffu, (v >> g) & 1u);
            if (lane == 0) gb[g * 4 + warp] = word;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        orv[(size_t)head * nt + tile] = so[0] | so[1] | so[2] | so[3];
        andv[(size_t)head * nt + tile] = sa[0] & sa[1] & sa[2] & sa[3];
    }
}

// Per KV head and group g: which key tiles hold a member of g (from the OR summaries) and which key tiles
// consist of members of g only (from the AND summaries), as bitmaps over the key tiles.  thread = (head, word).
__global__ void __launch_bounds__(256)
group_tiles_kernel(const uint32_t* __restrict__ ork, const uint32_t* __restrict__ andk, int HK, int nkt, int nkw, int K,
                   uint32_t* __restrict__ kany, uint32_t* __restrict__ kall) {
    const int gid = blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= HK * nkw) return;
    const int hk = gid / nkw, wd = gid % nkw;
    uint32_t any_w[32], all_w[32];
#pragma unroll
    for (int g = 0; g < 32; ++g) any_w[g] = all_w[g] = 0u;
    for (int c = 0; c < 32; ++c) {
        const int b = wd * 32 + c;
        if (b >= nkt) break;
        const uint32_t o = ork[(size_t)hk * nkt + b], a = andk[(size_t)hk * nkt + b];
#pragma unroll
        for (int g = 0; g < 32; ++g) {
            any_w[g] |= ((o >> g) & 1u) << c;
            all_w[g] |= ((a >> g) & 1u) << c;
        }
    }
    for (int g = 0; g < K; ++g) {
        kany[((size_t)hk * K + g) * nkw + wd] = any_w[g];
        kall[((size_t)hk * K + g) * nkw + wd] = all_w[g];
    }
}

// Live far-tile bitmap.  Key tile b is far for query tile a when every pair has i - j > w, i.e. b < (128 a - w) / 128;
// a far tile is live when the query tile's OR summary meets the key tile's, full when the AND summaries meet.  A word
// of the bitmap is the OR, over the groups present in the query tile, of the groups' key-tile bitmaps.
// One block per (query tile, head); threads stride over the words of the row.
__global__ void __launch_bounds__(128)
live_kernel(const uint32_t* __restrict__ orq, const uint32_t* __restrict__ andq, const uint32_t* __restrict__ kany,
            const uint32_t* __restrict__ kall, int G_heads, int Hq, int Hkv, int w, int K, int nqt, int nkw,
            uint32_t* __restrict__ live, int32_t* __restrict__ live_cnt, unsigned long long* counters) {
    const int a = blockIdx.x, hq = blockIdx.y;
    const int b_idx = hq / Hq, h = hq % Hq;
    const int hk = b_idx * Hkv + h / G_heads;
    const uint32_t oq = orq[(size_t)hq * nqt + a], aq = andq[(size_t)hq * nqt + a];
    const long long d = (long long)a * TM - w;
    const int nfar_tiles = d > 0 ? (int)(d / TN) : 0;                 // far tiles are the first nfar_tiles key tiles
    unsigned int nlive = 0, nfull = 0;
    for (int wd = threadIdx.x; wd < nkw; wd += blockDim.x) {
        const int rem = nfar_tiles - wd * 32;
        const uint32_t far_mask = rem >= 32 ? 0xffffffffu : (rem <= 0 ? 0u : ((1u << rem) - 1u));
        uint32_t lv = 0, fl = 0;
        if (far_mask) {
            for (uint32_t m = oq; m; m &= m - 1) {
                const int g = __ffs(m) - 1;
                if (g < K) lv |= kany[((size_t)hk * K + g) * nkw + wd];
            }
            for (uint32_t m = aq; m; m &= m - 1) {
                const int g = __ffs(m) - 1;
                if (g < K) fl |= kall[((size_t)hk * K + g) * nkw + wd];
            }
            lv &= far_mask;
            fl &= far_mask;
        }
        live[((size_t)hq * nqt + a) * nkw + wd] = lv;
        nlive += __popc(lv);
        nfull += __popc(fl);
    }
    __shared__ unsigned int s[2];
    if (threadIdx.x < 2) s[threadIdx.x] = 0;
    __syncthreads();
    if (nlive) atomicAdd(&s[0], nlive);
    if (nfull) atomicAdd(&s[1], nfull);
    __syncthreads();
    if (threadIdx.x == 0) {
        live_cnt[(size_t)hq * nqt + a] = (int32_t)s[0];
        if (nfar_tiles) atomicAdd(&counters[0], (unsigned long long)nfar_tiles);
        if (s[0]) atomicAdd(&counters[1], (unsigned long long)s[0]);
        if (s[1]) atomicAdd(&counters[2], (unsigned long long)s[1]);
    }
}

// Exact attended-pair count.  One block per (128-row query tile, head); thread = row.
// Row i keeps min(i, w) + 1 local keys plus every key j < i - w whose group bitmap bit is set in
// the OR of the bitmaps of the row's own groups.
__global__ void __launch_bounds__(128)
count_kept_kernel(const uint32_t* __restrict__ mq, const uint32_t* __restrict__ gbits, int G_heads, int Hq, int Hkv,
                  int n, int w, int K, int nkt, unsigned long long* __restrict__ out) {
    const int a = blockIdx.x, hq = blockIdx.y;
    const int b_idx = hq / Hq, h = hq % Hq;
    const int hk = b_idx * Hkv + h / G_heads;
    const int i = a * 128 + threadIdx.x;
    unsigned long long cnt = 0;
    if (i < n) {
        const uint32_t mi = mq[(size_t)hq * n + i];
        cnt = (unsigned long long)min(i, w) + 1ull;
        const long long nfar = (long long)i - w;            // keys 0 .. nfar-1 are beyond the window
        if (nfar > 0) {
            const int last_tile = (int)((nfar - 1) / TN);
            for (int b = 0; b <= last_tile; ++b) {
                const uint32_t* gb = gbits + ((size_t)hk * nkt + b) * K * 4;
                uint32_t wd[4] = {0, 0, 0, 0};
                uint32_t rem = mi;
                while (rem) {
                    const int g = __ffs(rem) - 1;
                    rem &= rem - 1;
                    if (g < K) {
                        const uint4 t = *reinterpret_cast<const uint4*>(gb + g * 4);
                        wd[0] |= t.x; wd[1] |= t.y; wd[2] |= t.z; wd[3] |= t.w;
                    }
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const long long lim = nfar - ((long long)b * TN + q * 32);   // keys of this word below lim are far
                    uint32_t valid = lim >= 32 ? 0xffffffffu : (lim <= 0 ? 0u : ((1u << (int)lim) - 1u));
                    cnt += __popc(wd[q] & valid);
                }
            }
        }
    }
    // block reduce
    for (int off = 16; off >= 1; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
    __shared__ unsigned long long s[4];
    if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = cnt;
    __syncthreads();
    if (threadIdx.x == 0) atomicAdd(&out[hq], s[0] + s[1] + s[2] + s[3]);
}

int launch_build_tiles_sorted(const focus_shape* s, const uint32_t* mq, const uint32_t* mk,
                              const focus_tiles_layout& L, char* ws, cudaStream_t st);

int launch_build_tiles(const focus_shape* s, const uint32_t* mq, const uint32_t* mk, int layout,
                       const focus_tiles_layout& L, char* ws, cudaStream_t st) {
    const int HQ = s->batch * s->Hq, HK = s->batch * s->Hkv;
    int rc = check_cuda(cudaMemsetAsync(ws + L.counters, 0, 8 * sizeof(uint64_t), st), "cudaMemsetAsync(counters)");
    if (rc) return rc;
    auto* orq = reinterpret_cast<uint32_t*>(ws + L.orq);
    auto* andq = reinterpret_cast<uint32_t*>(ws + L.andq);
    auto* ork = reinterpret_cast<uint32_t*>(ws + L.ork);
    auto* andk = reinterpret_cast<uint32_t*>(ws + L.andk);
    auto* gb = reinterpret_cast<uint32_t*>(ws + L.gbits);
    summarise_kernel<<<dim3(L.nqt, HQ), 128, 0, st>>>(mq, s->n, L.nqt, s->K, orq, andq, nullptr);
    summarise_kernel<<<dim3(L.nkt, HK), 128, 0, st>>>(mk, s->n, L.nkt, s->K, ork, andk, gb);
    auto* kany = reinterpret_cast<uint32_t*>(ws + L.kany);
    auto* kall = reinterpret_cast<uint32_t*>(ws + L.kall);
    group_tiles_kernel<<<cdiv(HK * L.nkw, 256), 256, 0, st>>>(ork, andk, HK, L.nkt, L.nkw, s->K, kany, kall);
    live_kernel<<<dim3(L.nqt, HQ), 128, 0, st>>>(orq, andq, kany, kall, s->Hq / s->Hkv, s->Hq, s->Hkv, s->window, s->K, L.nqt,
                                                 L.nkw, reinterpret_cast<uint32_t*>(ws + L.live),
                                                 reinterpret_cast<int32_t*>(ws + L.live_cnt),
                                                 reinterpret_cast<unsigned long long*>(ws + L.counters));
    if ((rc = check_cuda(cudaGetLastError(), "build_tiles kernels"))) return rc;
    if (layout_is_sorted(layout))
        return launch_build_tiles_sorted(s, mq, mk, L, ws, st);
    return FOCUS_OK;
}

int launch_count_kept(const focus_shape* s, const uint32_t* mq, const focus_tiles_layout& L, const char* ws,
                      unsigned long long* out, cudaStream_t st) {
    const int HQ = s->batch * s->Hq;
    int rc = check_cuda(cudaMemsetAsync(out, 0, (size_t)HQ * sizeof(unsigned long long), st), "cudaMemsetAsync(counts)");
    if (rc) return rc;
    count_kept_kernel<<<dim3(L.nqt, HQ), 128, 0, st>>>(mq, reinterpret_cast<const uint32_t*>(ws + L.gbits),
                                                       s->Hq / s->Hkv, s->Hq, s->Hkv, s->n, s->window, s->K, L.nkt, out);
    return check_cuda(cudaGetLastError(), "count_kept kernel");
}

}  // namespace focus
