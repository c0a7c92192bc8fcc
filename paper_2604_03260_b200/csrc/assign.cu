// focus_assign: cosine of every head vector with the K centroids of its KV head, top-k membership
// mask out (paper Eq. 1 + the top-k rule of Sec. 3.6).  HBM-bound: 2 D bytes read and 4 written per vector.
//
// The tiles of 128 vectors, numbered head by head, are dealt out as one contiguous range per block, a few blocks
// per SM and all of them resident, so the launch is a single wave of equal shares.  The rows of a tile go to
// shared memory with coalesced asynchronous 16-byte copies, laid out as the K-major, 128-byte-swizzled operand of
// a tcgen05 MMA, two tiles in flight (at D = 256 a tile travels as two pieces of 128 columns, so that three
// blocks still fit an SM); whenever its range enters a head with another centroid set the block splits
// those centroids into three bf16 terms each (hi + mid + lo carries 24 mantissa bits, so the products with the
// bf16 vectors sum to the fp32 dot product) as the second operand.  Per tile one thread issues the MMA chain S = X C'^T (128 x 3K, fp32, in tensor
// memory); while it runs every thread sums the squares of its own row from shared memory; then it reads its
// row of S, adds the three terms per group, scales by 1/(|x| |c_g|), selects the top-k groups and writes its
// mask word, while the copies of the tile after next are already under way.
#include "assign_common.cuh"
#include "sm100_ptx.cuh"

namespace focus {

using namespace ptx;

constexpr int ASSIGN_THREADS = 128;   // one thread per vector = one lane of tensor memory

template <int D, int KMAX>
struct AssignCfg {
    static constexpr int NCOLS = (3 * KMAX + 15) / 16 * 16;             // rows of C' = columns of S
    static constexpr uint32_t SUB_BYTES = 128 * 128;                     // 128 vectors x 64 dimensions
    static constexpr int CW = D < 128 ? D : 128;                         // columns of a tile staged at a time (a "piece")
    static constexpr int NP = D / CW;                                    // pieces per tile: 2 at D = 256
    static constexpr uint32_t TILE_BYTES = SUB_BYTES * (CW / 64);        // one piece of one tile
    static constexpr uint32_t CSUB_BYTES = NCOLS * 128;                  // NCOLS rows x 64 dimensions
    static constexpr uint32_t C_BYTES = CSUB_BYTES * (D / 64);
    static constexpr uint32_t TMEM_COLS2 = 2 * NCOLS <= 32 ? 32 : (2 * NCOLS <= 64 ? 64 : (2 * NCOLS <= 128 ? 128 : 256));   // two S buffers
    static constexpr uint32_t SMEM_BYTES = 2 * TILE_BYTES + C_BYTES + 256;
    static_assert(C_BYTES % 1024 == 0, "the vector tile and the centroid operand both start on a swizzle atom");
};

struct AssignCtl {
    uint64_t s_full[2];               // the MMAs that read the piece in buffer 0 / 1 have completed
    uint32_t tmem_base;
    int fault;
    float cn2[32];                    // |c_g|^2, then 1/|c_g|
};

template <int D, int KMAX>
__global__ void __launch_bounds__(ASSIGN_THREADS)
assign_kernel(const __nv_bfloat16* __restrict__ x, int64_t stride_b, int64_t stride_h, int64_t stride_n,
              int H, int G, int n, int K, int topk, int ntile, int share, int extra, const float* __restrict__ C,
              uint32_t* __restrict__ masks, unsigned long long* near_ties, float eps) {
    using Cfg = AssignCfg<D, KMAX>;
    extern __shared__ __align__(1024) unsigned char sm[];
    const uint32_t base = smem_u32(sm);
    const uint32_t sx = base;                                  // two vector tiles
    const uint32_t sc = base + 2 * Cfg::TILE_BYTES;            // centroid operand C'
    unsigned char* const cprime = sm + 2 * Cfg::TILE_BYTES;
    AssignCtl* const ctl = reinterpret_cast<AssignCtl*>(sm + 2 * Cfg::TILE_BYTES + Cfg::C_BYTES);
    constexpr int CW = Cfg::CW, NP = Cfg::NP;
    constexpr int CPR = CW / 8;                                // 16-byte chunks per row of a piece
    constexpr int RSTEP = ASSIGN_THREADS / CPR;                // rows covered by one copy per thread

    // block i takes `share` items, the first `extra` blocks one more: items item0 .. item0 + T - 1 of the list
    // (batch * head, tile), tile fastest
    const int item0 = blockIdx.x * share + min((int)blockIdx.x, extra);
    const int T = share + ((int)blockIdx.x < extra ? 1 : 0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // the swizzle is a function of the shared-memory address: a base off the 1024-byte grid would scramble both
    // operands, so such a block reports a fault and computes nothing
    const bool aligned = (base & 1023u) == 0;

    // ---- copies of one tile: consecutive threads copy consecutive chunks of a row, a thread's next copy is RSTEP rows
    // further down; rows past n are not copied (what their lanes compute is never written or counted).  Every call
    // commits one group, empty when the tile does not exist.
    const int r0 = threadIdx.x / CPR, cc = threadIdx.x % CPR;
    const __nv_bfloat16* const xrow0 = x + (size_t)r0 * stride_n + cc * 8;
    const size_t step = (size_t)RSTEP * stride_n;
    const uint32_t dst0 = sx + (cc >> 3) * Cfg::SUB_BYTES + r0 * 128;
    auto copy_tile = [&](int q) {                               // q = piece number: tile q / NP, columns (q % NP) * CW ...
        if (q < T * NP) {
            const int t = q / NP, c = q % NP;
            const int bh = (item0 + t) / ntile, tok0 = ((item0 + t) % ntile) * 128;
            const __nv_bfloat16* src = xrow0 + (size_t)(bh / H) * stride_b + (size_t)(bh % H) * stride_h + (size_t)tok0 * stride_n + c * CW;
            const int left = n - tok0 - r0;                    // copy i is in range iff i * RSTEP < left
            const uint32_t dstb = dst0 + (q & 1) * Cfg::TILE_BYTES;
#pragma unroll
            for (int i = 0; i < ASSIGN_THREADS / RSTEP; ++i) {
                const uint32_t dst = dstb + i * RSTEP * 128 + ((((uint32_t)cc & 7u) ^ ((uint32_t)(r0 + (i * RSTEP) % 8) & 7u)) << 4);
                if (i * RSTEP < left) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
                src += step;
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    copy_tile(0);
    copy_tile(1);
    if (warp == 0) {
        tmem_alloc(smem_u32(&ctl->tmem_base), Cfg::TMEM_COLS2);
        tmem_relinquish();
    }
    if (threadIdx.x == 32) {
        mbar_init(smem_u32(&ctl->s_full[0]), 1);
        mbar_init(smem_u32(&ctl->s_full[1]), 1);
        fence_mbar_init();
        ctl->fault = 0;
    }
    __syncthreads();

    // ---- C': the centroids of KV head hk, each split into hi + mid + lo (rows g, KMAX + g, 2 KMAX + g); the rest zero.
    // Called by the whole block between tiles: every MMA that read the previous C' has completed, and the first
    // barrier keeps the previous norms until every thread has used them.
    auto build_centroids = [&](int hk) {
        __syncthreads();
        if (threadIdx.x < 32) ctl->cn2[threadIdx.x] = 0.f;
        __syncthreads();
        const float* Ch = C + (size_t)hk * K * D;
#pragma unroll
        for (int j = 0; j < KMAX * D / ASSIGN_THREADS; ++j) {
            const int e = j * ASSIGN_THREADS + threadIdx.x;
            const int g = e / D, d = e % D;                     // g is the same for the 32 lanes of a warp (D >= 64)
            float v = g < K ? __ldg(Ch + e) : 0.f;
            float s = v * v;
            __nv_bfloat16 hi, mid, lo;
            split3_bf16(v, hi, mid, lo);
            *reinterpret_cast<__nv_bfloat16*>(cprime + sw128_offset(g, d, Cfg::NCOLS)) = hi;
            *reinterpret_cast<__nv_bfloat16*>(cprime + sw128_offset(KMAX + g, d, Cfg::NCOLS)) = mid;
            *reinterpret_cast<__nv_bfloat16*>(cprime + sw128_offset(2 * KMAX + g, d, Cfg::NCOLS)) = lo;
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
            if (lane == 0) atomicAdd(&ctl->cn2[g], s);
        }
        constexpr int ZROWS = Cfg::NCOLS - 3 * KMAX;           // whole rows, so the swizzle does not matter for them
        if constexpr (ZROWS > 0) {
            for (int i = threadIdx.x; i < ZROWS * (D / 64) * 8; i += ASSIGN_THREADS) {
                const int sub = i / (ZROWS * 8), rem = i % (ZROWS * 8);
                *reinterpret_cast<uint4*>(cprime + sub * Cfg::CSUB_BYTES + (3 * KMAX) * 128 + rem * 16) = make_uint4(0, 0, 0, 0);
            }
        }
        __syncthreads();
        if (threadIdx.x < KMAX) {
            const float s = ctl->cn2[threadIdx.x];
            ctl->cn2[threadIdx.x] = s > 0.f ? rsqrtf(s) : 0.f;  // read by everyone after the tile's first barrier
        }
    };

    bool ok = aligned;
    uint32_t tmem = 0;
    unsigned int near_votes = 0;
    int cur_hk = -1;
    float2 a0 = make_float2(0.f, 0.f), a1 = make_float2(0.f, 0.f);      // |x|^2 of the thread's row, over the pieces
    for (int q = 0; q < T * NP; ++q) {
        const int t = q / NP, c = q % NP;                      // tile and piece
        const int buf = q & 1, abuf = t & 1;                   // piece buffer, accumulator buffer
        const int bh = (item0 + t) / ntile, tile = (item0 + t) % ntile;
        const int hk = (bh % H) / G;
        if (hk != cur_hk) {
            build_centroids(hk);
            cur_hk = hk;
        }
        asm volatile("cp.async.wait_group 1;" ::: "memory");   // this thread's copies of tile t have landed
        fence_proxy_async_smem();                              // generic-proxy writes before the MMA's async-proxy reads
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        tmem = ctl->tmem_base;
        if (warp == 0) {
            if (aligned && elect_one()) {
                constexpr uint32_t IDESC = idesc_bf16(128, Cfg::NCOLS, 0, 0);
                const uint64_t xd = smem_desc_sw128(sx + buf * Cfg::TILE_BYTES, 16, 1024);
                const uint64_t cd = smem_desc_sw128(sc, 16, 1024);
#pragma unroll
                for (int ks = 0; ks < CW / 16; ++ks)
                    umma_ss(tmem + abuf * Cfg::NCOLS, xd + (uint64_t)(((ks / 4) * Cfg::SUB_BYTES + (ks % 4) * 32) >> 4),
                            cd + (uint64_t)(((c * (CW / 64) + ks / 4) * Cfg::CSUB_BYTES + (ks % 4) * 32) >> 4), IDESC,
                            (c > 0 || ks > 0) ? 1u : 0u);
                umma_commit(smem_u32(&ctl->s_full[buf]));
            }
            __syncwarp();
        }
        // ---- |x|^2 of the thread's own row while the MMAs run (packed fp32 pairs)
        {
            const unsigned char* row = sm + buf * Cfg::TILE_BYTES + threadIdx.x * 128;
            const uint32_t sw = (threadIdx.x & 7u) << 4;
            if (c == 0) a0 = a1 = make_float2(0.f, 0.f);
#pragma unroll
            for (int v = 0; v < CPR; ++v) {
                const uint4 rv = *reinterpret_cast<const uint4*>(row + (v >> 3) * Cfg::SUB_BYTES + ((((uint32_t)v & 7u) << 4) ^ sw));
                const float2 v0 = make_float2(__uint_as_float(rv.x << 16), __uint_as_float(rv.x & 0xffff0000u));
                const float2 v1 = make_float2(__uint_as_float(rv.y << 16), __uint_as_float(rv.y & 0xffff0000u));
                const float2 v2 = make_float2(__uint_as_float(rv.z << 16), __uint_as_float(rv.z & 0xffff0000u));
                const float2 v3 = make_float2(__uint_as_float(rv.w << 16), __uint_as_float(rv.w & 0xffff0000u));
                a0 = __ffma2_rn(v0, v0, a0); a1 = __ffma2_rn(v1, v1, a1);
                a0 = __ffma2_rn(v2, v2, a0); a1 = __ffma2_rn(v3, v3, a1);
            }
        }
        const float xx = (a0.x + a0.y) + (a1.x + a1.y);
        const bool last_piece = c == NP - 1;
        if (ok && !mbar_wait(smem_u32(&ctl->s_full[buf]), (uint32_t)((q >> 1) & 1))) {
            ok = false;
            ctl->fault = 1;
        }
        tc_fence_after();
        float sc3[Cfg::NCOLS];
        if (ok && last_piece) {
#pragma unroll
            for (int cc16 = 0; cc16 < Cfg::NCOLS / 16; ++cc16) {
                uint32_t v[16];
                tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + abuf * Cfg::NCOLS + cc16 * 16, v);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 16; ++e) sc3[cc16 * 16 + e] = __uint_as_float(v[e]);
            }
        } else {
#pragma unroll
            for (int e = 0; e < Cfg::NCOLS; ++e) sc3[e] = 0.f;
        }
        tc_fence_before();
        __syncthreads();                                       // the piece's buffer is free: its MMAs and every row sum are done
        copy_tile(q + 2);
        if (!last_piece) continue;

        const int tok = tile * 128 + threadIdx.x;
        const bool in = tok < n;
        const float xinv = xx > 0.f ? rsqrtf(xx) : 0.f;
        float cosv[KMAX];
#pragma unroll
        for (int g = 0; g < KMAX; ++g) cosv[g] = ((sc3[2 * KMAX + g] + sc3[KMAX + g]) + sc3[g]) * ctl->cn2[g] * xinv;
        float last, next;
        const uint32_t taken = select_topk<KMAX>(cosv, K, topk, last, next);
        if (in && ok) masks[(size_t)bh * n + tok] = taken;
        if (near_ties) near_votes += __popc(__ballot_sync(0xffffffffu, ok && in && topk < K && (last - next) < eps));
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (near_ties && lane == 0 && near_votes) atomicAdd(near_ties, (unsigned long long)near_votes);
    __syncthreads();
    if (warp == 0) {
        if (ctl->fault || !aligned) {
            if (lane == 0 && near_ties) atomicOr(near_ties, 1ull << 63);
            const uint64_t t0 = globaltimer_ns();
            while (globaltimer_ns() - t0 < 20000ull) { }       // MMAs already issued finish before the columns go back
        }
        tmem_dealloc(ctl->tmem_base, Cfg::TMEM_COLS2);
    }
}

template <int D, int KMAX>
static int launch_one(const focus_shape* s, const focus_tensor& x, int H, const float* C, uint32_t* masks,
                      unsigned long long* near_ties, float eps, cudaStream_t st) {
    using Cfg = AssignCfg<D, KMAX>;
    auto kern = assign_kernel<D, KMAX>;
    int rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::SMEM_BYTES),
                        "cudaFuncSetAttribute(assign)");
    if (rc) return rc;
    if ((rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, 100), "cudaFuncSetAttribute(assign)"))) return rc;
    // one resident wave: as many blocks as fit on the device at once (fewer when there are fewer tiles).  Blocks of
    // 128 threads per SM: by shared memory (227 KB, 1 KB reserved per block), by the 512 columns of tensor memory, and
    // at most 4 (64 K registers, up to 128 per thread)
    int dev = 0, sms = 0;
    if ((rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice"))) return rc;
    if ((rc = check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "cudaDeviceGetAttribute"))) return rc;
    int per_sm = (int)(227 * 1024 / (Cfg::SMEM_BYTES + 1024));
    if (per_sm > (int)(512 / Cfg::TMEM_COLS2)) per_sm = (int)(512 / Cfg::TMEM_COLS2);
    if (per_sm > 4) per_sm = 4;
    if (per_sm < 1) per_sm = 1;
    const long long resident = (long long)sms * per_sm;
    const int ntile = cdiv(s->n, 128);
    const long long nitems = (long long)s->batch * H * ntile;
    if (nitems > 0x7fffffffll) return fail(FOCUS_ERR_UNSUPPORTED, "focus_assign: %lld tiles of 128 vectors exceed 2^31 - 1", nitems);
    if (nitems == 0) return 0;
    const int nblocks = (int)(nitems < resident ? nitems : resident);
    const int share = (int)(nitems / nblocks), extra = (int)(nitems % nblocks);
    kern<<<nblocks, ASSIGN_THREADS, Cfg::SMEM_BYTES, st>>>(reinterpret_cast<const __nv_bfloat16*>(x.ptr), x.stride_b, x.stride_h,
                                                           x.stride_n, H, H / s->Hkv, s->n, s->K, s->topk, ntile, share, extra, C, masks,
                                                           near_ties, eps);
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
