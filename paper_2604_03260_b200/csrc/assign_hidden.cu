// focus_assign_hidden: the router as the paper states it (Sec. 2 "Learned grouping", Eq. 1): one
// routing vector per token, W_g h_i in d_g dimensions, scored against the centroids by dot product;
// the token joins its top-k groups and every head (query and key role alike) uses that mask.
//
// W_g^T h . C_g = h . (W_g C_g), so the projection and the centroids fold into K vectors of length d
// (a small kernel, once per call); scoring then reads each hidden state exactly once, which makes the
// pass HBM-bound: 2 d bytes per token.
//
// Scoring runs on the tensor cores.  The tiles of 128 tokens are dealt out as one contiguous range per block,
// one resident wave of small blocks.  A block walks its tiles in chunks of 128 elements of d: the chunk of the
// 128 rows goes to shared memory with coalesced asynchronous 16-byte copies, laid out as the K-major,
// 128-byte-swizzled operand of a tcgen05 MMA, in a ring of three stages (a stage is refilled as soon as the
// MMAs of the chunk before the current one are done, so two chunks are in flight while a third is multiplied);
// the same chunk of the K folded vectors (loaded into registers one chunk ahead) is
// split into three bf16 terms each (hi + mid + lo carries 24 mantissa bits, so the products with the bf16 hidden
// states sum to the fp32 dot product) as the second operand.  One thread issues the MMAs of the chunk, which
// accumulate S = H F'^T (128 x 3K, fp32) in tensor memory over the chunks of the tile; after the last chunk every
// thread reads its row of S, adds the three terms per group and the bias, and selects (or stores the scores).
#include "assign_common.cuh"
#include "sm100_ptx.cuh"

namespace focus {

using namespace ptx;

constexpr int AH_THREADS = 128;      // one thread per token of the tile = one lane of tensor memory
constexpr int AH_CHUNK = 128;        // elements of d per stage: two 64-column sub-tiles
constexpr int AH_NS = 3;             // stages of the chunk ring: one being read by the MMAs, two being filled

template <int KMAX>
struct HiddenCfg {
    static constexpr int NCOLS = (3 * KMAX + 15) / 16 * 16;             // rows of F' = columns of S
    static constexpr uint32_t SUB_BYTES = 128 * 128;                     // 128 tokens x 64 elements
    static constexpr uint32_t A_BYTES = (AH_CHUNK / 64) * SUB_BYTES;
    static constexpr uint32_t FSUB_BYTES = NCOLS * 128;                  // NCOLS rows x 64 elements
    static constexpr uint32_t F_BYTES = (AH_CHUNK / 64) * FSUB_BYTES;
    static constexpr uint32_t STAGE_BYTES = A_BYTES + F_BYTES;
    static constexpr uint32_t TMEM_COLS = NCOLS <= 32 ? 32 : (NCOLS <= 64 ? 64 : 128);
    static constexpr uint32_t SMEM_BYTES = AH_NS * STAGE_BYTES + 256;
    static_assert(STAGE_BYTES % 1024 == 0, "every operand starts on a swizzle atom");
};

struct HiddenCtl {
    uint64_t mma_done[AH_NS];         // the MMAs that read the stage have completed
    uint32_t tmem_base;
    int fault;
};

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
                     float* __restrict__ scores, int ntile, int share, int extra) {
    using Cfg = HiddenCfg<KMAX>;
    extern __shared__ __align__(1024) unsigned char sm[];
    const uint32_t base = smem_u32(sm);
    HiddenCtl* const ctl = reinterpret_cast<HiddenCtl*>(sm + AH_NS * Cfg::STAGE_BYTES);
    constexpr int CPR = AH_CHUNK / 8;                          // 16-byte pieces per row of a chunk
    constexpr int RSTEP = AH_THREADS / CPR;                    // rows covered by one copy per thread (8)

    // block i takes `share` tiles, the first `extra` blocks one more: tiles item0 .. item0 + T - 1 of the list
    // (batch, tile); its work is the T * nchunk chunks of those tiles, walked in order
    const int item0 = blockIdx.x * share + min((int)blockIdx.x, extra);
    const int T = share + ((int)blockIdx.x < extra ? 1 : 0);
    const int nchunk = (d + AH_CHUNK - 1) / AH_CHUNK;
    const int total = T * nchunk;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // the swizzle is a function of the shared-memory address: a base off the 1024-byte grid would scramble both
    // operands, so such a block reports a fault and computes nothing
    const bool aligned = (base & 1023u) == 0;

    // ---- stage one chunk: rows by asynchronous copies (consecutive threads copy consecutive pieces of a row, a
    // thread's next copy is 8 rows further down; rows past n are not copied: what their lanes compute is never
    // written or counted; pieces past d are zero), folded vectors split on the way in (thread = column).  Every
    // call commits one group, empty when the chunk does not exist.  (it, ic) = tile and chunk of the next call.
    const int r0 = threadIdx.x / CPR, cc = threadIdx.x % CPR;
    int it_next = 0, ic_next = 0;
    constexpr int FPT = KMAX * AH_CHUNK / AH_THREADS;          // folded values per thread and chunk
    float fv[FPT];                                             // those of the chunk the next call stages, loaded one call ahead
    auto load_folded = [&]() {
        const int e0 = ic_next * AH_CHUNK;
#pragma unroll
        for (int i = 0; i < FPT; ++i) {
            const int q = i * AH_THREADS + threadIdx.x;
            const int g = q / AH_CHUNK, e = e0 + q % AH_CHUNK;
            fv[i] = (g < K && e < d) ? __ldg(folded + (size_t)g * d + e) : 0.f;
        }
    };
    load_folded();
    auto stage_chunk = [&](int j) {
        if (j < total) {
            const int item = item0 + it_next;
            const int b = item / ntile, tok0 = (item % ntile) * 128;
            const int e0 = ic_next * AH_CHUNK;
            unsigned char* const st = sm + (j % AH_NS) * Cfg::STAGE_BYTES;
            const uint32_t dstb = base + (j % AH_NS) * Cfg::STAGE_BYTES + (cc >> 3) * Cfg::SUB_BYTES + r0 * 128 +
                                  ((((uint32_t)cc & 7u) ^ ((uint32_t)r0 & 7u)) << 4);
            if (e0 + cc * 8 < d) {
                const __nv_bfloat16* src = h + (size_t)b * stride_b + (size_t)(tok0 + r0) * stride_n + e0 + cc * 8;
                const size_t step = (size_t)RSTEP * stride_n;
                const int left = n - tok0 - r0;                // copy i is in range iff i * RSTEP < left
#pragma unroll
                for (int i = 0; i < AH_THREADS / RSTEP; ++i) {
                    if (i * RSTEP < left)
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dstb + i * RSTEP * 128), "l"(src) : "memory");
                    src += step;
                }
            } else {
#pragma unroll
                for (int i = 0; i < AH_THREADS / RSTEP; ++i)
                    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dstb + i * RSTEP * 128), "r"(0) : "memory");
            }
            unsigned char* const fp = st + Cfg::A_BYTES;
#pragma unroll
            for (int i = 0; i < FPT; ++i) {
                const int q = i * AH_THREADS + threadIdx.x;
                const int g = q / AH_CHUNK, col = q % AH_CHUNK;
                __nv_bfloat16 hi, mid, lo;
                split3_bf16(fv[i], hi, mid, lo);
                *reinterpret_cast<__nv_bfloat16*>(fp + sw128_offset(g, col, Cfg::NCOLS)) = hi;
                *reinterpret_cast<__nv_bfloat16*>(fp + sw128_offset(KMAX + g, col, Cfg::NCOLS)) = mid;
                *reinterpret_cast<__nv_bfloat16*>(fp + sw128_offset(2 * KMAX + g, col, Cfg::NCOLS)) = lo;
            }
            if (++ic_next == nchunk) { ic_next = 0; ++it_next; }
            if (j + 1 < total) load_folded();
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    // rows of F' beyond 3 KMAX stay zero in both stages (whole rows, so the swizzle does not matter for them)
    {
        constexpr int ZROWS = Cfg::NCOLS - 3 * KMAX;
        if constexpr (ZROWS > 0) {
            constexpr int NSUB = AH_CHUNK / 64;
            for (int i = threadIdx.x; i < AH_NS * NSUB * ZROWS * 8; i += AH_THREADS) {
                const int stg = i / (NSUB * ZROWS * 8), rem = i % (NSUB * ZROWS * 8);
                const int sub = rem / (ZROWS * 8), q = rem % (ZROWS * 8);
                *reinterpret_cast<uint4*>(sm + stg * Cfg::STAGE_BYTES + Cfg::A_BYTES + sub * Cfg::FSUB_BYTES + (3 * KMAX) * 128 + q * 16) =
                    make_uint4(0, 0, 0, 0);
            }
        }
    }
#pragma unroll
    for (int j = 0; j < AH_NS - 1; ++j) stage_chunk(j);
    if (warp == 0) {
        tmem_alloc(smem_u32(&ctl->tmem_base), Cfg::TMEM_COLS);
        tmem_relinquish();
    }
    if (threadIdx.x == 32) {
        for (int i = 0; i < AH_NS; ++i) mbar_init(smem_u32(&ctl->mma_done[i]), 1);
        fence_mbar_init();
        ctl->fault = 0;
    }

    bool ok = aligned;
    unsigned int near_votes = 0;
    int it = 0, ic = 0;                                        // tile and chunk of iteration j
    for (int j = 0; j < total; ++j) {
        const int buf = j % AH_NS;
        asm volatile("cp.async.wait_group %0;" ::"n"(AH_NS - 2) : "memory");   // this thread's copies of chunk j have landed
        fence_proxy_async_smem();                              // generic-proxy writes before the MMA's async-proxy reads
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        const uint32_t tmem = ctl->tmem_base;
        if (warp == 0) {
            if (aligned && elect_one()) {
                constexpr uint32_t IDESC = idesc_bf16(128, Cfg::NCOLS, 0, 0);
                const uint64_t ad = smem_desc_sw128(base + buf * Cfg::STAGE_BYTES, 16, 1024);
                const uint64_t fd = smem_desc_sw128(base + buf * Cfg::STAGE_BYTES + Cfg::A_BYTES, 16, 1024);
#pragma unroll
                for (int ks = 0; ks < AH_CHUNK / 16; ++ks)
                    umma_ss(tmem, ad + (uint64_t)(((ks / 4) * Cfg::SUB_BYTES + (ks % 4) * 32) >> 4),
                            fd + (uint64_t)(((ks / 4) * Cfg::FSUB_BYTES + (ks % 4) * 32) >> 4), IDESC, (ic > 0 || ks > 0) ? 1u : 0u);
                umma_commit(smem_u32(&ctl->mma_done[buf]));
            }
            __syncwarp();
        }
        // the stage chunk j - 1 was read from is free once its MMAs are done (long ago, as a rule): refill it while
        // the MMAs of chunk j run
        if (ok && j > 0 && !mbar_wait(smem_u32(&ctl->mma_done[(j - 1) % AH_NS]), (uint32_t)(((j - 1) / AH_NS) & 1))) {
            ok = false;
            ctl->fault = 1;
        }
        stage_chunk(j + AH_NS - 1);
        const bool last_chunk = ic == nchunk - 1;
        float sc3[Cfg::NCOLS];
        if (last_chunk) {
            if (ok && !mbar_wait(smem_u32(&ctl->mma_done[buf]), (uint32_t)((j / AH_NS) & 1))) {
                ok = false;
                ctl->fault = 1;
            }
            tc_fence_after();
            if (ok) {
#pragma unroll
                for (int c = 0; c < Cfg::NCOLS / 16; ++c) {
                    uint32_t v[16];
                    tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + c * 16, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 16; ++e) sc3[c * 16 + e] = __uint_as_float(v[e]);
                }
            } else {
#pragma unroll
                for (int e = 0; e < Cfg::NCOLS; ++e) sc3[e] = 0.f;
            }
            tc_fence_before();
        }

        if (last_chunk) {
            const int item = item0 + it;
            const int b = item / ntile, tok = (item % ntile) * 128 + threadIdx.x;
            const bool in = tok < n;
            float score[KMAX];
#pragma unroll
            for (int g = 0; g < KMAX; ++g)
                score[g] = ((sc3[2 * KMAX + g] + sc3[KMAX + g]) + sc3[g]) + ((bias && g < K) ? __ldg(bias + g) : 0.f);
            if (scores) {   // the scores themselves (training-time soft assignment), rows of KMAX floats, zero beyond K
                if (in && ok) {
                    float4* o = reinterpret_cast<float4*>(scores + ((size_t)b * n + tok) * KMAX);
#pragma unroll
                    for (int c = 0; c < KMAX / 4; ++c)
                        o[c] = make_float4(4 * c < K ? score[4 * c] : 0.f, 4 * c + 1 < K ? score[4 * c + 1] : 0.f,
                                           4 * c + 2 < K ? score[4 * c + 2] : 0.f, 4 * c + 3 < K ? score[4 * c + 3] : 0.f);
                }
            } else {
                float last, next;
                const uint32_t taken = select_topk<KMAX>(score, K, topk, last, next);
                if (in && ok) {   // every head of the layer shares the token's mask
                    if (mq) for (int hh = 0; hh < Hq; ++hh) mq[((size_t)b * Hq + hh) * n + tok] = taken;
                    if (mk) for (int hh = 0; hh < Hkv; ++hh) mk[((size_t)b * Hkv + hh) * n + tok] = taken;
                }
                if (near_ties) near_votes += __popc(__ballot_sync(0xffffffffu, ok && in && topk < K && (last - next) < eps));
            }
        }
        if (++ic == nchunk) { ic = 0; ++it; }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (near_ties && lane == 0 && near_votes) atomicAdd(near_ties, (unsigned long long)near_votes);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        if (ctl->fault || !aligned) {
            if (lane == 0 && near_ties) atomicOr(near_ties, 1ull << 63);
            const uint64_t t0 = globaltimer_ns();
            while (globaltimer_ns() - t0 < 20000ull) { }       // MMAs already issued finish before the columns go back
        }
        tmem_dealloc(ctl->tmem_base, Cfg::TMEM_COLS);
    }
}

template <int KMAX>
static int launch_k(const focus_shape* s, const void* h, int64_t sb, int64_t sn, int d, const float* folded, const float* bias,
                    uint32_t* mq, uint32_t* mk, unsigned long long* near_ties, float eps, float* scores, cudaStream_t st) {
    using Cfg = HiddenCfg<KMAX>;
    auto kern = assign_hidden_kernel<KMAX>;
    int rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::SMEM_BYTES),
                        "cudaFuncSetAttribute(assign_hidden)");
    if (rc) return rc;
    if ((rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, 100),
                         "cudaFuncSetAttribute(assign_hidden)"))) return rc;
    // one resident wave: as many blocks as fit on the device at once (fewer when there are fewer tiles).  Blocks of
    // 128 threads per SM: by shared memory (227 KB, 1 KB reserved per block), by the 512 columns of tensor memory, at most 3
    int dev = 0, sms = 0;
    if ((rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice"))) return rc;
    if ((rc = check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "cudaDeviceGetAttribute"))) return rc;
    int per_sm = (int)(227 * 1024 / (Cfg::SMEM_BYTES + 1024));
    if (per_sm > (int)(512 / Cfg::TMEM_COLS)) per_sm = (int)(512 / Cfg::TMEM_COLS);
    if (per_sm > 3) per_sm = 3;
    if (per_sm < 1) per_sm = 1;
    const long long resident = (long long)sms * per_sm;
    const int ntile = cdiv(s->n, 128);
    const long long nitems = (long long)s->batch * ntile;
    if (nitems == 0) return 0;
    if (nitems > 0x7fffffffll || (long long)(nitems / (nitems < resident ? nitems : resident) + 1) * cdiv(d, AH_CHUNK) > 0x7fffffffll)
        return fail(FOCUS_ERR_UNSUPPORTED, "focus_assign_hidden: too many chunks of 128 x 128 elements for one launch");
    const int nblocks = (int)(nitems < resident ? nitems : resident);
    const int share = (int)(nitems / nblocks), extra = (int)(nitems % nblocks);
    kern<<<nblocks, AH_THREADS, Cfg::SMEM_BYTES, st>>>(reinterpret_cast<const __nv_bfloat16*>(h), sb, sn, s->n, d, s->K, s->topk, folded,
                                                       bias, s->Hq, s->Hkv, mq, mk, near_ties, eps, scores, ntile, share, extra);
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
