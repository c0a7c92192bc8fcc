// Class-sorted layout of focus_build_tiles (paper Sec. 2, item "Group": sort tokens by group with a
// stable sort, which keeps causal order inside a group).
//
// A token's class is its membership-mask value.  Per head the tokens are stably sorted by class
// (classes ascending by mask value, original positions ascending inside a class); every class
// segment is padded to a whole number of tiles, so that a tile of the sorted order holds one class.
// Then a (query tile, key tile) pair is all-share or none-share, and the attended pairs of a query
// block are: for every key class that shares a group with the block's class, the keys of that class
// up to the block's last position; for every other key class, only the keys inside the window.
// These ranges are written per block of 256 sorted queries, together with an order of the blocks
// (most key tiles first inside each KV head group) for the persistent attention kernel.
#include "common.cuh"

#include <limits.h>

namespace focus {

constexpr int MAXC = FOCUS_MAX_CLASSES;
constexpr unsigned long long HASH_EMPTY = 0ull;

__device__ __forceinline__ unsigned int hash_slot(uint32_t v) { return (v * 2654435761u) >> 24; }   // 0..255

// ---------------------------------------------------------------------------------------------
// 1. distinct mask values per head: block-local hash set, merged into a global one per head
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
collect_classes_kernel(const uint32_t* __restrict__ m, int n, unsigned long long* __restrict__ table) {
    __shared__ unsigned long long loc[SORT_HASH];
    const int head = blockIdx.y;
    for (int s = threadIdx.x; s < SORT_HASH; s += blockDim.x) loc[s] = HASH_EMPTY;
    __syncthreads();
    const int t0 = blockIdx.x * SORT_CHUNK;
    for (int t = t0 + threadIdx.x; t < min(n, t0 + SORT_CHUNK); t += blockDim.x) {
        const uint32_t v = m[(size_t)head * n + t];
        const unsigned long long key = (1ull << 32) | v;
        unsigned int s = hash_slot(v);
        for (int probe = 0; probe < SORT_HASH; ++probe) {
            const unsigned long long old = atomicCAS(&loc[s], HASH_EMPTY, key);
            if (old == HASH_EMPTY || old == key) break;
            s = (s + 1) & (SORT_HASH - 1);
        }
    }
    __syncthreads();
    unsigned long long* glob = table + (size_t)head * SORT_HASH;
    for (int i = threadIdx.x; i < SORT_HASH; i += blockDim.x) {
        const unsigned long long key = loc[i];
        if (key == HASH_EMPTY) continue;
        unsigned int s = hash_slot((uint32_t)key);
        for (int probe = 0; probe < SORT_HASH; ++probe) {
            const unsigned long long old = atomicCAS(&glob[s], HASH_EMPTY, key);
            if (old == HASH_EMPTY || old == key) break;
            s = (s + 1) & (SORT_HASH - 1);
        }
    }
}

// one block per head: compact the hash set, sort ascending, flag more than MAXC values
__global__ void __launch_bounds__(SORT_HASH)
finalize_classes_kernel(const unsigned long long* __restrict__ table, uint32_t* __restrict__ cls,
                        int32_t* __restrict__ ncls, unsigned long long* counters) {
    __shared__ uint32_t vals[SORT_HASH];
    __shared__ int cnt;
    const int head = blockIdx.x;
    if (threadIdx.x == 0) cnt = 0;
    __syncthreads();
    const unsigned long long key = table[(size_t)head * SORT_HASH + threadIdx.x];
    if (key != HASH_EMPTY) vals[atomicAdd(&cnt, 1)] = (uint32_t)key;
    __syncthreads();
    const int c = cnt;
    if (threadIdx.x < c) {
        const uint32_t v = vals[threadIdx.x];
        int rank = 0;
        for (int j = 0; j < c; ++j) rank += vals[j] < v;
        if (rank < MAXC) cls[(size_t)head * MAXC + rank] = v;
    }
    if (threadIdx.x == 0) {
        ncls[head] = min(c, MAXC);
        if (c > MAXC) atomicAdd(&counters[4], 1ull);
    }
}

// index of value v in the ascending table (values not in the table, possible only after an
// overflow, fall into the last class below them)
__device__ __forceinline__ int class_index(const uint32_t* tab, int c, uint32_t v) {
    int lo = 0, hi = c - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (tab[mid] <= v) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// ---------------------------------------------------------------------------------------------
// 2. counting sort: per-chunk histograms, scan over chunks, stable scatter
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(SORT_CHUNK)
chunk_hist_kernel(const uint32_t* __restrict__ m, int n, const uint32_t* __restrict__ cls,
                  const int32_t* __restrict__ ncls, int nchunk, int32_t* __restrict__ hist) {
    __shared__ uint32_t tab[MAXC];
    __shared__ int h[MAXC];
    const int head = blockIdx.y, chunk = blockIdx.x;
    if (threadIdx.x < MAXC) { tab[threadIdx.x] = cls[(size_t)head * MAXC + threadIdx.x]; h[threadIdx.x] = 0; }
    __syncthreads();
    const int c = ncls[head];
    const int t = chunk * SORT_CHUNK + threadIdx.x;
    if (t < n) atomicAdd(&h[class_index(tab, c, m[(size_t)head * n + t])], 1);
    __syncthreads();
    if (threadIdx.x < MAXC) hist[((size_t)head * nchunk + chunk) * MAXC + threadIdx.x] = h[threadIdx.x];
}

// one block of MAXC threads per head (thread = class): running offsets over the chunks, class
// totals and padded segment starts
__global__ void __launch_bounds__(MAXC)
scan_chunks_kernel(int32_t* __restrict__ hist, int nchunk, const int32_t* __restrict__ ncls, int pad,
                   int32_t* __restrict__ cnt, int32_t* __restrict__ seg, int npad, unsigned long long* counters) {
    __shared__ int tot[MAXC];
    const int head = blockIdx.x, c = threadIdx.x;
    int run = 0;
    for (int k = 0; k < nchunk; ++k) {
        int32_t* p = hist + ((size_t)head * nchunk + k) * MAXC + c;
        const int v = *p;
        *p = run;                   // tokens of class c in earlier chunks
        run += v;
    }
    tot[c] = run;
    cnt[(size_t)head * MAXC + c] = run;
    __syncthreads();
    if (c == 0) {
        const int nc = ncls[head];
        int s = 0;
        for (int j = 0; j <= MAXC; ++j) {
            seg[(size_t)head * (MAXC + 1) + j] = s;
            if (j < nc) s += (tot[j] + pad - 1) / pad * pad;
        }
        if (s > npad) atomicAdd(&counters[4], 1ull);      // more entries than the sorted arrays hold (group-major lists of
                                                          // masks with more than topk bits): the attention kernel refuses
    }
}

__global__ void fill_kernel(int32_t* __restrict__ p, size_t count, int32_t value) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (size_t)gridDim.x * blockDim.x)
        p[i] = value;
}

// stable scatter: slot = segment start + tokens of the class in earlier chunks + earlier warps of
// this chunk + earlier lanes of this warp
__global__ void __launch_bounds__(SORT_CHUNK)
scatter_kernel(const uint32_t* __restrict__ m, int n, const uint32_t* __restrict__ cls, const int32_t* __restrict__ ncls,
               int nchunk, const int32_t* __restrict__ base, const int32_t* __restrict__ seg, int npad,
               int32_t* __restrict__ perm) {
    __shared__ uint32_t tab[MAXC];
    __shared__ int wcnt[SORT_CHUNK / 32][MAXC];
    const int head = blockIdx.y, chunk = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x < MAXC) tab[threadIdx.x] = cls[(size_t)head * MAXC + threadIdx.x];
    for (int i = threadIdx.x; i < (SORT_CHUNK / 32) * MAXC; i += blockDim.x) (&wcnt[0][0])[i] = 0;
    __syncthreads();
    const int c = ncls[head];
    const int t = chunk * SORT_CHUNK + threadIdx.x;
    const bool in = t < n;
    const int ci = in ? class_index(tab, c, m[(size_t)head * n + t]) : -1;
    const unsigned int same = __match_any_sync(0xffffffffu, ci);
    const int rank = __popc(same & ((1u << lane) - 1u));
    if (in && rank == 0) wcnt[warp][ci] = __popc(same);
    __syncthreads();
    if (threadIdx.x < MAXC) {               // exclusive scan over the warps, per class
        int run = 0;
        for (int w = 0; w < SORT_CHUNK / 32; ++w) {
            const int v = wcnt[w][threadIdx.x];
            wcnt[w][threadIdx.x] = run;
            run += v;
        }
    }
    __syncthreads();
    if (in) {
        const int slot = seg[(size_t)head * (MAXC + 1) + ci] + base[((size_t)head * nchunk + chunk) * MAXC + ci] +
                         wcnt[warp][ci] + rank;
        if (slot < npad) perm[(size_t)head * npad + slot] = t;
    }
}

// ---------------------------------------------------------------------------------------------
// 2b. group-major keys: K lists per KV head, list g = the keys that are members of group g, in token order.
// "Class" j of the key side is group j, so that the range and attention code reads the lists like class segments.
// ---------------------------------------------------------------------------------------------
__global__ void group_classes_kernel(int heads, int K, uint32_t* __restrict__ cls, int32_t* __restrict__ ncls) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < heads * MAXC) cls[i] = (i % MAXC) < K ? 1u << (i % MAXC) : 0u;
    if (i < heads) ncls[i] = K;
}

__global__ void __launch_bounds__(SORT_CHUNK)
group_hist_kernel(const uint32_t* __restrict__ m, int n, int K, int nchunk, int32_t* __restrict__ hist) {
    __shared__ int h[MAXC];
    const int head = blockIdx.y, chunk = blockIdx.x;
    if (threadIdx.x < MAXC) h[threadIdx.x] = 0;
    __syncthreads();
    const int t = chunk * SORT_CHUNK + threadIdx.x;
    const uint32_t v = t < n ? m[(size_t)head * n + t] : 0u;
    for (int g = 0; g < K; ++g) {
        const unsigned int b = __ballot_sync(0xffffffffu, (v >> g) & 1u);
        if ((threadIdx.x & 31) == 0 && b) atomicAdd(&h[g], __popc(b));
    }
    __syncthreads();
    if (threadIdx.x < MAXC) hist[((size_t)head * nchunk + chunk) * MAXC + threadIdx.x] = h[threadIdx.x];
}

// stable scatter into the lists: a key goes to the list of every group it belongs to
__global__ void __launch_bounds__(SORT_CHUNK)
group_scatter_kernel(const uint32_t* __restrict__ m, int n, int K, int nchunk, const int32_t* __restrict__ base,
                     const int32_t* __restrict__ seg, int npad, int32_t* __restrict__ perm) {
    __shared__ int wcnt[SORT_CHUNK / 32][32];
    const int head = blockIdx.y, chunk = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = chunk * SORT_CHUNK + threadIdx.x;
    const uint32_t v = t < n ? m[(size_t)head * n + t] : 0u;
    int rank[32];
#pragma unroll
    for (int g = 0; g < 32; ++g) {
        const unsigned int b = g < K ? __ballot_sync(0xffffffffu, (v >> g) & 1u) : 0u;
        rank[g] = __popc(b & ((1u << lane) - 1u));
        if (lane == 0) wcnt[warp][g] = __popc(b);
    }
    __syncthreads();
    if (threadIdx.x < 32) {                 // exclusive scan over the warps, per group
        int run = 0;
        for (int w = 0; w < SORT_CHUNK / 32; ++w) {
            const int c = wcnt[w][threadIdx.x];
            wcnt[w][threadIdx.x] = run;
            run += c;
        }
    }
    __syncthreads();
#pragma unroll
    for (int g = 0; g < 32; ++g) {
        if (g < K && ((v >> g) & 1u)) {
            const int slot = seg[(size_t)head * (MAXC + 1) + g] + base[((size_t)head * nchunk + chunk) * MAXC + g] +
                             wcnt[warp][g] + rank[g];
            if (slot < npad) perm[(size_t)head * npad + slot] = t;
        }
    }
}

// block of 128 threads per (tile of the lists, KV head): per group the bitmap of entries that are members of it
__global__ void __launch_bounds__(128)
gbits_sorted_kernel(const uint32_t* __restrict__ m, int n, int K, const int32_t* __restrict__ perm, int npad,
                    uint32_t* __restrict__ gbits_s) {
    const int tile = blockIdx.x, head = blockIdx.y;
    const int pos = perm[(size_t)head * npad + (size_t)tile * 128 + threadIdx.x];
    const uint32_t v = (pos >= 0 && pos < n) ? m[(size_t)head * n + pos] : 0u;
    uint32_t* gb = gbits_s + ((size_t)head * (npad / 128) + tile) * K * 4;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int g = 0; g < K; ++g) {
        const uint32_t word = __ballot_sync(0xffffffffu, (v >> g) & 1u);
        if (lane == 0) gb[g * 4 + warp] = word;
    }
}

// ---------------------------------------------------------------------------------------------
// 3. key-tile ranges per query block, block costs, block order
// ---------------------------------------------------------------------------------------------
// number of entries of the ascending array a[0..len) that are <= v
__device__ __forceinline__ int count_le(const int32_t* __restrict__ a, int len, long long v) {
    int lo = 0, hi = len;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if ((long long)a[mid] <= v) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// thread = (query head, query block, key class)
__global__ void __launch_bounds__(256)
qrange_kernel(int HQ, int Hq, int Hkv, int G_heads, int w, int nqp, int nkp, const int32_t* __restrict__ ncls_q,
              const int32_t* __restrict__ ncls_k, const uint32_t* __restrict__ cls_q, const uint32_t* __restrict__ cls_k,
              const int32_t* __restrict__ cnt_q, const int32_t* __restrict__ cnt_k, const int32_t* __restrict__ seg_q,
              const int32_t* __restrict__ seg_k, const int32_t* __restrict__ perm_q, const int32_t* __restrict__ perm_k,
              int32_t* __restrict__ qrange, int32_t* __restrict__ cost, unsigned long long* counters, int sharing_only) {
    const int nqblk = nqp / 256;
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= (long long)HQ * nqblk * MAXC) return;
    const int jk = (int)(gid % MAXC);
    const int blk = (int)((gid / MAXC) % nqblk);
    const int hq = (int)(gid / ((long long)MAXC * nqblk));
    const int hk = (hq / Hq) * Hkv + (hq % Hq) / G_heads;
    int first = 0, last = 0;
    const int32_t* sq = seg_q + (size_t)hq * (MAXC + 1);
    const int ncq = ncls_q[hq], nck = ncls_k[hk];
    const int start = blk * 256;
    if (jk < nck && start < sq[ncq]) {
        int jq = 0;
        while (jq + 1 < ncq && sq[jq + 1] <= start) ++jq;          // class of this query block
        const int valid_end = sq[jq] + cnt_q[(size_t)hq * MAXC + jq];    // one past the last real row of the class
        const int32_t* pq = perm_q + (size_t)hq * nqp;
        const long long pmin = pq[start], pmax = pq[min(start + 256, valid_end) - 1];
        const int ks0 = seg_k[(size_t)hk * (MAXC + 1) + jk], kc = cnt_k[(size_t)hk * MAXC + jk];
        const int32_t* pk = perm_k + (size_t)hk * nkp + ks0;
        const bool share = (cls_q[(size_t)hq * MAXC + jq] & cls_k[(size_t)hk * MAXC + jk]) != 0u;
        const int hi = count_le(pk, kc, pmax);                             // keys at or before the block's last position
        const int lo = share ? 0 : count_le(pk, kc, pmin - w - 1);          // keys before the window of the first row
        // with a separate window pass only the classes that share a group with the block's class are listed
        if (hi > lo && (share || !sharing_only)) {
            first = (ks0 + lo) / 128;
            last = (ks0 + hi + 127) / 128;
        }
    }
    qrange[gid * 2] = first;
    qrange[gid * 2 + 1] = last;
    if (last > first) {
        atomicAdd(&cost[(size_t)hq * nqblk + blk], last - first);
        atomicAdd(&counters[3], (unsigned long long)(last - first));
    }
}

// one block per KV head group: counting sort of its (query head, query block) pairs by cost, descending
constexpr int ORDER_BUCKETS = 2048;
__global__ void __launch_bounds__(1024)
order_kernel(int Hq, int Hkv, int G_heads, int nqblk, int max_cost, const int32_t* __restrict__ cost,
             int32_t* __restrict__ order) {
    __shared__ int bucket[ORDER_BUCKETS];
    __shared__ int carry;
    const int grp = blockIdx.x;                          // batch * Hkv + KV head
    const int hq0 = (grp / Hkv) * Hq + (grp % Hkv) * G_heads;
    const int items = G_heads * nqblk;
    for (int i = threadIdx.x; i < ORDER_BUCKETS; i += blockDim.x) bucket[i] = 0;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    auto bucket_of = [&](int c) {                        // bucket 0 holds the most expensive blocks
        long long q = (long long)c * (ORDER_BUCKETS - 1) / (max_cost > 0 ? max_cost : 1);
        if (q > ORDER_BUCKETS - 1) q = ORDER_BUCKETS - 1;
        return ORDER_BUCKETS - 1 - (int)q;
    };
    for (int i = threadIdx.x; i < items; i += blockDim.x) {
        const int g = i / nqblk, blk = i % nqblk;
        atomicAdd(&bucket[bucket_of(cost[(size_t)(hq0 + g) * nqblk + blk])], 1);
    }
    __syncthreads();
    // exclusive scan of the buckets, 1024 at a time
    for (int b0 = 0; b0 < ORDER_BUCKETS; b0 += 1024) {
        const int idx = b0 + threadIdx.x;
        const int v = bucket[idx];
        int x = v;
        // inclusive scan inside the warp, then across warps through shared memory
        for (int off = 1; off < 32; off <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, x, off);
            if ((threadIdx.x & 31) >= off) x += y;
        }
        __shared__ int wsum[32];
        if ((threadIdx.x & 31) == 31) wsum[threadIdx.x >> 5] = x;
        __syncthreads();
        if (threadIdx.x < 32) {
            int s = wsum[threadIdx.x];
            for (int off = 1; off < 32; off <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, s, off);
                if (threadIdx.x >= off) s += y;
            }
            wsum[threadIdx.x] = s;
        }
        __syncthreads();
        const int before = carry + (threadIdx.x >= 32 ? wsum[(threadIdx.x >> 5) - 1] : 0) + x - v;
        __syncthreads();
        bucket[idx] = before;
        if (threadIdx.x == 1023) carry = before + v;
        __syncthreads();
    }
    int32_t* out = order + (size_t)grp * items * 2;
    for (int i = threadIdx.x; i < items; i += blockDim.x) {
        const int g = i / nqblk, blk = i % nqblk;
        const int pos = atomicAdd(&bucket[bucket_of(cost[(size_t)(hq0 + g) * nqblk + blk])], 1);
        out[2 * pos] = hq0 + g;
        out[2 * pos + 1] = blk;
    }
}

// ---------------------------------------------------------------------------------------------
// 4. gather of Q / K / V rows into the sorted order (run by focus_attn_fwd), 16 bytes per thread
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
gather_rows_kernel(const __nv_bfloat16* __restrict__ src, int64_t sb, int64_t sh, int64_t sn, int H, int D,
                   const int32_t* __restrict__ perm, const int32_t* __restrict__ seg, int npad, int n,
                   __nv_bfloat16* __restrict__ dst) {
    const int vec = D / 8;                               // 16-byte vectors per row
    const int head = blockIdx.y;
    const int used = seg[(size_t)head * (MAXC + 1) + MAXC];
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int slot = (int)(gid / vec), v = (int)(gid % vec);
    if (slot >= used) return;
    const int pos = perm[(size_t)head * npad + slot];
    uint4 val = make_uint4(0u, 0u, 0u, 0u);              // padding rows are zero
    if (pos >= 0 && pos < n) {
        const __nv_bfloat16* row = src + (size_t)(head / H) * sb + (size_t)(head % H) * sh + (size_t)pos * sn;
        val = *reinterpret_cast<const uint4*>(row + v * 8);
    }
    *reinterpret_cast<uint4*>(dst + ((size_t)head * npad + slot) * D + v * 8) = val;
}

int launch_gather_sorted(const focus_shape* s, const focus_tensor& t, int H, bool query, const focus_tiles_layout& L,
                         const char* ws, char* dst, cudaStream_t st) {
    const int heads = s->batch * H;
    const int npad = query ? L.nqp : L.nkp;
    const long long threads = (long long)npad * (s->D / 8);
    gather_rows_kernel<<<dim3((unsigned)((threads + 255) / 256), heads), 256, 0, st>>>(
        reinterpret_cast<const __nv_bfloat16*>(t.ptr), t.stride_b, t.stride_h, t.stride_n, H, s->D,
        reinterpret_cast<const int32_t*>(ws + (query ? L.perm_q : L.perm_k)),
        reinterpret_cast<const int32_t*>(ws + (query ? L.seg_q : L.seg_k)), npad, s->n,
        reinterpret_cast<__nv_bfloat16*>(dst));
    return check_cuda(cudaGetLastError(), "gather kernel");
}

// ---------------------------------------------------------------------------------------------
int launch_build_tiles_sorted(const focus_shape* s, const uint32_t* mq, const uint32_t* mk,
                              const focus_tiles_layout& L, char* ws, cudaStream_t st) {
    const int HQ = s->batch * s->Hq, HK = s->batch * s->Hkv;
    const int nchunk = cdiv(s->n, SORT_CHUNK);
    const int nqblk = L.nqp / 256;
    // scratch: hash sets | chunk histograms | block costs
    char* scr = ws + L.scratch;
    auto* table = reinterpret_cast<unsigned long long*>(scr);
    const size_t table_bytes = align_up((size_t)(HQ + HK) * SORT_HASH * 8, 256);
    auto* hist = reinterpret_cast<int32_t*>(scr + table_bytes);
    const size_t hist_bytes = align_up((size_t)(HQ + HK) * nchunk * MAXC * 4, 256);
    auto* cost = reinterpret_cast<int32_t*>(scr + table_bytes + hist_bytes);
    const size_t cost_bytes = (size_t)HQ * nqblk * 4;
    auto* counters = reinterpret_cast<unsigned long long*>(ws + L.counters);
    int rc;
    if ((rc = check_cuda(cudaMemsetAsync(table, 0, table_bytes, st), "cudaMemsetAsync(class tables)"))) return rc;
    if ((rc = check_cuda(cudaMemsetAsync(cost, 0, cost_bytes, st), "cudaMemsetAsync(block costs)"))) return rc;
    if ((rc = check_cuda(cudaMemsetAsync(ws + L.cls_q, 0, (size_t)HQ * MAXC * 4, st), "cudaMemsetAsync(cls_q)"))) return rc;
    if ((rc = check_cuda(cudaMemsetAsync(ws + L.cls_k, 0, (size_t)HK * MAXC * 4, st), "cudaMemsetAsync(cls_k)"))) return rc;

    for (int side = 0; side < 2; ++side) {
        const int heads = side ? HK : HQ;
        const uint32_t* m = side ? mk : mq;
        unsigned long long* tab = table + (side ? (size_t)HQ * SORT_HASH : 0);
        int32_t* hs = hist + (side ? (size_t)HQ * nchunk * MAXC : 0);
        auto* cls = reinterpret_cast<uint32_t*>(ws + (side ? L.cls_k : L.cls_q));
        auto* ncls = reinterpret_cast<int32_t*>(ws + (side ? L.ncls_k : L.ncls_q));
        auto* cnt = reinterpret_cast<int32_t*>(ws + (side ? L.cnt_k : L.cnt_q));
        auto* seg = reinterpret_cast<int32_t*>(ws + (side ? L.seg_k : L.seg_q));
        auto* perm = reinterpret_cast<int32_t*>(ws + (side ? L.perm_k : L.perm_q));
        const int npad = side ? L.nkp : L.nqp;
        if (side && L.layout == FOCUS_LAYOUT_GROUP_MAJOR) {
            group_classes_kernel<<<cdiv(heads * MAXC, 256), 256, 0, st>>>(heads, s->K, cls, ncls);
            group_hist_kernel<<<dim3(nchunk, heads), SORT_CHUNK, 0, st>>>(m, s->n, s->K, nchunk, hs);
            scan_chunks_kernel<<<heads, MAXC, 0, st>>>(hs, nchunk, ncls, 128, cnt, seg, npad, counters);
            fill_kernel<<<1184, 256, 0, st>>>(perm, (size_t)heads * npad, INT_MAX);
            group_scatter_kernel<<<dim3(nchunk, heads), SORT_CHUNK, 0, st>>>(m, s->n, s->K, nchunk, hs, seg, npad, perm);
            gbits_sorted_kernel<<<dim3(npad / 128, heads), 128, 0, st>>>(m, s->n, s->K, perm, npad,
                                                                         reinterpret_cast<uint32_t*>(ws + L.gbits_s));
            continue;
        }
        collect_classes_kernel<<<dim3(nchunk, heads), 256, 0, st>>>(m, s->n, tab);
        finalize_classes_kernel<<<heads, SORT_HASH, 0, st>>>(tab, cls, ncls, counters);
        chunk_hist_kernel<<<dim3(nchunk, heads), SORT_CHUNK, 0, st>>>(m, s->n, cls, ncls, nchunk, hs);
        scan_chunks_kernel<<<heads, MAXC, 0, st>>>(hs, nchunk, ncls, side ? 128 : 256, cnt, seg, npad, counters);
        fill_kernel<<<1184, 256, 0, st>>>(perm, (size_t)heads * npad, side ? INT_MAX : -1);
        scatter_kernel<<<dim3(nchunk, heads), SORT_CHUNK, 0, st>>>(m, s->n, cls, ncls, nchunk, hs, seg, npad, perm);
    }
    const long long nthreads = (long long)HQ * nqblk * MAXC;
    qrange_kernel<<<(unsigned)((nthreads + 255) / 256), 256, 0, st>>>(
        HQ, s->Hq, s->Hkv, s->Hq / s->Hkv, s->window, L.nqp, L.nkp, reinterpret_cast<const int32_t*>(ws + L.ncls_q),
        reinterpret_cast<const int32_t*>(ws + L.ncls_k), reinterpret_cast<const uint32_t*>(ws + L.cls_q),
        reinterpret_cast<const uint32_t*>(ws + L.cls_k), reinterpret_cast<const int32_t*>(ws + L.cnt_q),
        reinterpret_cast<const int32_t*>(ws + L.cnt_k), reinterpret_cast<const int32_t*>(ws + L.seg_q),
        reinterpret_cast<const int32_t*>(ws + L.seg_k), reinterpret_cast<const int32_t*>(ws + L.perm_q),
        reinterpret_cast<const int32_t*>(ws + L.perm_k), reinterpret_cast<int32_t*>(ws + L.qrange), cost, counters,
        layout_has_window_pass(L.layout) ? 1 : 0);
    order_kernel<<<HK, 1024, 0, st>>>(s->Hq, s->Hkv, s->Hq / s->Hkv, nqblk, L.nkp / 128, cost,
                                      reinterpret_cast<int32_t*>(ws + L.order));
    return check_cuda(cudaGetLastError(), "build_tiles (class-sorted) kernels");
}

// ---- FOCUS_LAYOUT_SORTED_LOCAL: the two partial results (sharing pairs from the class-sorted pass, window-only pairs
// from the pass in token order) cover disjoint sets of pairs and join through their logsumexps (paper Appendix D).

__global__ void __launch_bounds__(256) fill_f32_kernel(float* __restrict__ x, size_t count, float v) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) x[i] = v;
}

int launch_fill_f32(float* x, size_t count, float v, cudaStream_t st) {
    fill_f32_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(x, count, v);
    return check_cuda(cudaGetLastError(), "fill kernel launch");
}

// thread = 8 consecutive elements of a row; the D/8 threads of a row sit in one warp, so that all of them have read the
// row's two logsumexps before the first of them overwrites one
template <int D>
__global__ void __launch_bounds__(256)
merge_partials_kernel(__nv_bfloat16* __restrict__ o, int64_t o_sb, int64_t o_sh, int64_t o_sn, float* __restrict__ lse,
                      const float* __restrict__ o_sorted, const float* __restrict__ o_local, const float* __restrict__ lse_local,
                      int Hq, int n) {
    constexpr int TPR = D / 8;
    const int hq = blockIdx.y;
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long i = t / TPR;
    const int c = (int)(t % TPR);
    const bool in = i < n;
    float ls = -INFINITY, ll = -INFINITY;
    if (in) {
        ls = lse[(size_t)hq * n + i];
        ll = lse_local[(size_t)hq * n + i];
    }
    __syncwarp();
    if (!in) return;
    const float m = fmaxf(ls, ll);
    const float ws = m == -INFINITY ? 0.f : __expf(ls - m), wl = m == -INFINITY ? 0.f : __expf(ll - m);
    const float tot = ws + wl;
    const float inv = tot > 0.f ? 1.f / tot : 0.f;
    const size_t src = ((size_t)hq * n + i) * D + c * 8;
    float r[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) r[e] = 0.f;
    // a partial result without any pair has weight 0 and unspecified contents: it is not read
    if (ws > 0.f) {
        const float4 a0 = *reinterpret_cast<const float4*>(o_sorted + src), a1 = *reinterpret_cast<const float4*>(o_sorted + src + 4);
        const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
#pragma unroll
        for (int e = 0; e < 8; ++e) r[e] = av[e] * ws;
    }
    if (wl > 0.f) {
        const float4 b0 = *reinterpret_cast<const float4*>(o_local + src), b1 = *reinterpret_cast<const float4*>(o_local + src + 4);
        const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
        for (int e = 0; e < 8; ++e) r[e] = fmaf(bv[e], wl, r[e]);
    }
    uint32_t rw[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const __nv_bfloat162 h2 = __floats2bfloat162_rn(r[2 * e] * inv, r[2 * e + 1] * inv);
        rw[e] = *reinterpret_cast<const uint32_t*>(&h2);
    }
    __nv_bfloat16* orow = o + (size_t)(hq / Hq) * o_sb + (size_t)(hq % Hq) * o_sh + (size_t)i * o_sn + c * 8;
    *reinterpret_cast<uint4*>(orow) = make_uint4(rw[0], rw[1], rw[2], rw[3]);
    if (c == 0) lse[(size_t)hq * n + i] = tot > 0.f ? m + __logf(tot) : -INFINITY;
}

int launch_merge_partials(const focus_shape* s, const focus_tensor& o, float* lse, const float* o_sorted, const float* o_local,
                          const float* lse_local, cudaStream_t st) {
    const int HQ = s->batch * s->Hq;
    const long long threads = (long long)s->n * (s->D / 8);
    const dim3 grid((unsigned)((threads + 255) / 256), HQ);
    auto* op = reinterpret_cast<__nv_bfloat16*>(o.ptr);
    switch (s->D) {
        case 64: merge_partials_kernel<64><<<grid, 256, 0, st>>>(op, o.stride_b, o.stride_h, o.stride_n, lse, o_sorted, o_local, lse_local, s->Hq, s->n); break;
        case 128: merge_partials_kernel<128><<<grid, 256, 0, st>>>(op, o.stride_b, o.stride_h, o.stride_n, lse, o_sorted, o_local, lse_local, s->Hq, s->n); break;
        case 256: merge_partials_kernel<256><<<grid, 256, 0, st>>>(op, o.stride_b, o.stride_h, o.stride_n, lse, o_sorted, o_local, lse_local, s->Hq, s->n); break;
        default: return fail(FOCUS_ERR_UNSUPPORTED, "D (%d) must be 64, 128 or 256", s->D);
    }
    return check_cuda(cudaGetLastError(), "merge kernel launch");
}

}  // namespace focus
