// focus_selftest_umma: one 128 x 128 x D tile of S = A B^T (both operands from shared memory,
// K-major) and one 128 x D x 128 tile of O = P V (P from tensor memory, V from shared memory,
// MN-major), through the same TMA / descriptor / tcgen05 building blocks as the attention kernel.
// A diagnostic for the descriptor encodings; not on the hot path.
#include "common.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.cuh"

namespace focus {

template <int D>
__global__ void __launch_bounds__(128)
umma_selftest_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                     const __grid_constant__ CUtensorMap tm_v, const uint32_t* __restrict__ p_bits, float* s_out,
                     float* o_out, int32_t* status) {
    using namespace ptx;
    constexpr int SUBT = D / 64;
    constexpr uint32_t SUB_BYTES = 128 * 64 * 2;
    constexpr uint32_t TILE_BYTES = SUB_BYTES * SUBT;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sa = base, sb = base + TILE_BYTES, sv = base + 2 * TILE_BYTES;
    __shared__ __align__(8) uint64_t bars[2];
    __shared__ uint32_t tmem_base_s;
    const uint32_t bar_tma = smem_u32(&bars[0]), bar_mma = smem_u32(&bars[1]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(bar_tma, 1);
        mbar_init(bar_mma, 1);
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    constexpr uint32_t COL_S = 0, COL_P = 128, COL_O = 256;

    if (threadIdx.x == 0) {
        mbar_arrive_expect_tx(bar_tma, 3 * TILE_BYTES);
        for (int c = 0; c < SUBT; ++c) {
            tma_load_4d(sa + c * SUB_BYTES, &tm_a, bar_tma, c * 64, 0, 0, 0);
            tma_load_4d(sb + c * SUB_BYTES, &tm_b, bar_tma, c * 64, 0, 0, 0);
            tma_load_4d(sv + c * SUB_BYTES, &tm_v, bar_tma, c * 64, 0, 0, 0);
        }
    }
    // every thread writes its row of P (128 bf16 = 64 packed words) into tensor memory
    {
        const uint32_t* prow = p_bits + (size_t)threadIdx.x * 64;
        uint32_t r[32];
#pragma unroll
        for (int half = 0; half < 2; ++half) {
#pragma unroll
            for (int c = 0; c < 32; ++c) r[c] = prow[half * 32 + c];
            tmem_st32(tmem + lane_base + COL_P + half * 32, r);
        }
        tmem_wait_st();
    }
    tc_fence_before();
    __syncthreads();
    bool ok = true;
    if (warp == 0) {
        if (lane == 0) {
            tc_fence_after();
            ok = mbar_wait(bar_tma, 0);
            if (ok) {
                // S = A B^T : M = 128, N = 128, K = D in steps of 16
                constexpr uint32_t idesc_s = idesc_bf16(128, 128, 0, 0);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = (ks / 4) * SUB_BYTES + (ks % 4) * 32;
                    umma_ss(tmem + COL_S, smem_desc_sw128(sa + off, 16, 1024), smem_desc_sw128(sb + off, 16, 1024),
                            idesc_s, ks > 0);
                }
                // O = P V : M = 128, N = D, K = 128 keys in steps of 16; V is MN-major (D contiguous)
                constexpr uint32_t idesc_o = idesc_bf16(128, D, 0, 1);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    umma_ts(tmem + COL_O, tmem + COL_P + ks * 8, smem_desc_sw128(sv + ks * 2048, SUB_BYTES, 1024),
                            idesc_o, ks > 0);
                umma_commit(bar_mma);
            } else {
                atomicExch(status, 1);
                mbar_arrive(bar_mma);
            }
        }
        __syncwarp();
    }
    ok = mbar_wait(bar_mma, 0);
    tc_fence_after();
    if (!ok) atomicExch(status, 2);
    if (ok) {
        uint32_t r[32];
        for (int c = 0; c < 4; ++c) {
            tmem_ld32(tmem + lane_base + COL_S + c * 32, r);
            tmem_wait_ld();
            for (int e = 0; e < 32; ++e) s_out[(size_t)threadIdx.x * 128 + c * 32 + e] = __uint_as_float(r[e]);
        }
        for (int c = 0; c < D / 32; ++c) {
            tmem_ld32(tmem + lane_base + COL_O + c * 32, r);
            tmem_wait_ld();
            for (int e = 0; e < 32; ++e) o_out[(size_t)threadIdx.x * D + c * 32 + e] = __uint_as_float(r[e]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

template <int D>
static int run_selftest(const void* a, const void* b, const void* p, const void* v, float* s_out, float* o_out,
                        int32_t* status, cudaStream_t st) {
    CUtensorMap ta, tb, tv;
    int rc;
    if ((rc = make_tmap_bf16_4d(&ta, a, D, 128, 1, 1, D * 2, (uint64_t)D * 2 * 128, (uint64_t)D * 2 * 128, 64, 128))) return rc;
    if ((rc = make_tmap_bf16_4d(&tb, b, D, 128, 1, 1, D * 2, (uint64_t)D * 2 * 128, (uint64_t)D * 2 * 128, 64, 128))) return rc;
    if ((rc = make_tmap_bf16_4d(&tv, v, D, 128, 1, 1, D * 2, (uint64_t)D * 2 * 128, (uint64_t)D * 2 * 128, 64, 128))) return rc;
    const size_t smem = 3 * (size_t)128 * D * 2 + 1024;
    auto kern = umma_selftest_kernel<D>;
    if ((rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem),
                         "cudaFuncSetAttribute(selftest)")))
        return rc;
    kern<<<1, 128, smem, st>>>(ta, tb, tv, reinterpret_cast<const uint32_t*>(p), s_out, o_out, status);
    return check_cuda(cudaGetLastError(), "selftest launch");
}


// The same two tiles through one MMA shared by a pair of CTAs (cluster of two, cta_group::2), D = 128:
// S = A B^T with 256 rows (128 per CTA) and each CTA staging 64 of the 128 rows of B; O = P V with P in each CTA's
// own tensor memory and each CTA staging 64 of the 128 columns of V.  Every load is a plain TMA copy into the loading
// CTA's own shared memory that completes on the leader's mbarrier; the leader's commits go to one mbarrier per CTA.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(128)
umma_pair_selftest_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                          const __grid_constant__ CUtensorMap tm_v, const uint32_t* __restrict__ p_bits, float* s_out,
                          float* o_out, int32_t* status) {
    using namespace ptx;
    constexpr int D = 128;
    constexpr uint32_t A_BYTES = 128 * D * 2, BH_BYTES = 64 * D * 2, VH_BYTES = 128 * 64 * 2;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sa = base, sb = base + A_BYTES, sv = sb + BH_BYTES;
    __shared__ __align__(8) uint64_t bars[3];
    __shared__ uint32_t tmem_base_s;
    const uint32_t bar_tma = smem_u32(&bars[0]), bar_p = smem_u32(&bars[1]), bar_mma = smem_u32(&bars[2]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();

    if (threadIdx.x == 0) {
        mbar_init(bar_tma, 1);
        mbar_init(bar_p, 2);
        mbar_init(bar_mma, 1);
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc_pair(smem_u32(&tmem_base_s), 512);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                 // the other CTA's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    constexpr uint32_t COL_S = 0, COL_P = 128, COL_O = 256;

    if (threadIdx.x == 0) {
        if (rank == 0) mbar_arrive_expect_tx(bar_tma, 2 * (A_BYTES + BH_BYTES + VH_BYTES));
        const uint32_t lead_tma = mapa_shared(bar_tma, 0);
        for (int c = 0; c < 2; ++c) {
            tma_load_4d_pair(sa + c * (A_BYTES / 2), &tm_a, lead_tma, c * 64, (int)rank * 128, 0, 0);     // its 128 rows of A
            tma_load_4d_pair(sb + c * (BH_BYTES / 2), &tm_b, lead_tma, c * 64, (int)rank * 64, 0, 0);     // its 64 rows of B
        }
        tma_load_4d_pair(sv, &tm_v, lead_tma, (int)rank * 64, 0, 0, 0);                                  // its 64 columns of V
    }
    {   // every thread writes its row of P into its CTA's tensor memory
        const uint32_t* prow = p_bits + ((size_t)rank * 128 + threadIdx.x) * 64;
        uint32_t r[32];
#pragma unroll
        for (int half = 0; half < 2; ++half) {
#pragma unroll
            for (int c = 0; c < 32; ++c) r[c] = prow[half * 32 + c];
            tmem_st32(tmem + lane_base + COL_P + half * 32, r);
        }
        tmem_wait_st();
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) mbar_arrive_cluster(mapa_shared(bar_p, 0));
    if (rank == 0 && warp == 0) {
        if (lane == 0) {
            auto wait_cluster = [&](uint32_t bar) {
                const uint64_t t0 = globaltimer_ns();
                while (!mbar_try_wait_cluster(bar, 0))
                    if (globaltimer_ns() - t0 > 2000000000ull) return false;
                return true;
            };
            const bool ok = wait_cluster(bar_tma) && wait_cluster(bar_p);
            tc_fence_after();
            if (ok) {
                constexpr uint32_t idesc_s = idesc_bf16(256, 128, 0, 0);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    umma_ss_pair(tmem + COL_S, smem_desc_sw128(sa + (ks / 4) * (A_BYTES / 2) + (ks % 4) * 32, 16, 1024),
                                 smem_desc_sw128(sb + (ks / 4) * (BH_BYTES / 2) + (ks % 4) * 32, 16, 1024), idesc_s, ks > 0);
                constexpr uint32_t idesc_o = idesc_bf16(256, D, 0, 1);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    umma_ts_pair(tmem + COL_O, tmem + COL_P + ks * 8, smem_desc_sw128(sv + ks * 2048, VH_BYTES, 1024), idesc_o,
                                 ks > 0);
                umma_commit_pair(bar_mma);
                umma_commit_pair(mapa_shared(bar_mma, 1));
            } else {
                atomicExch(status, 1);
                mbar_arrive(bar_mma);
                mbar_arrive_cluster(mapa_shared(bar_mma, 1));
            }
        }
        __syncwarp();
    }
    const bool done = mbar_wait(bar_mma, 0, 3000000000ull);
    tc_fence_after();
    if (!done) atomicExch(status, 2);
    if (done && *(volatile int32_t*)status == 0) {
        uint32_t r[32];
        const size_t row = (size_t)rank * 128 + threadIdx.x;
        for (int c = 0; c < 4; ++c) {
            tmem_ld32(tmem + lane_base + COL_S + c * 32, r);
            tmem_wait_ld();
            for (int e = 0; e < 32; ++e) s_out[row * 128 + c * 32 + e] = __uint_as_float(r[e]);
        }
        for (int c = 0; c < D / 32; ++c) {
            tmem_ld32(tmem + lane_base + COL_O + c * 32, r);
            tmem_wait_ld();
            for (int e = 0; e < 32; ++e) o_out[row * D + c * 32 + e] = __uint_as_float(r[e]);
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                 // neither CTA leaves (or frees tensor memory) while the other may still use it
    if (warp == 0) tmem_dealloc_pair(tmem, 512);
}

static int run_pair_selftest(const void* a, const void* b, const void* p, const void* v, float* s_out, float* o_out,
                             int32_t* status, cudaStream_t st) {
    constexpr int D = 128;
    CUtensorMap ta, tb, tv;
    int rc;
    if ((rc = make_tmap_bf16_4d(&ta, a, D, 256, 1, 1, D * 2, (uint64_t)D * 2 * 256, (uint64_t)D * 2 * 256, 64, 128))) return rc;
    if ((rc = make_tmap_bf16_4d(&tb, b, D, 128, 1, 1, D * 2, (uint64_t)D * 2 * 128, (uint64_t)D * 2 * 128, 64, 64))) return rc;
    if ((rc = make_tmap_bf16_4d(&tv, v, D, 128, 1, 1, D * 2, (uint64_t)D * 2 * 128, (uint64_t)D * 2 * 128, 64, 128))) return rc;
    const size_t smem = (size_t)(128 * D * 2 + 64 * D * 2 + 128 * 64 * 2) + 1024;
    auto kern = umma_pair_selftest_kernel;
    if ((rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem),
                         "cudaFuncSetAttribute(pair selftest)")))
        return rc;
    kern<<<2, 128, smem, st>>>(ta, tb, tv, reinterpret_cast<const uint32_t*>(p), s_out, o_out, status);
    return check_cuda(cudaGetLastError(), "pair selftest launch");
}


// ---- focus_selftest_mma_rate: what the tensor pipe delivers when it is fed nothing but MMAs, in the shapes the attention
// kernel uses or could use.  One CTA (or CTA pair) per SM, operands resident in shared and tensor memory (pseudo-random
// finite bf16 values, so that the datapath switches as on real data), chains of eight K = 16 instructions (one
// 128 x N x 128 product, or 256 x N x 128 across a pair).  `pattern` 0: one chain per commit, two commits in flight;
// 1: two S-type chains per commit, issued alternately; 2: an S-type and a P V-type chain per commit, issued alternately;
// 3: an S-type chain, then a P V-type chain, per commit (four chains in flight in patterns 1-3).
template <int PAIR, int TS, int PATTERN>
__global__ void __launch_bounds__(128) mma_rate_kernel(int N, int rounds, unsigned long long* res) {
    constexpr int ts = TS, pattern = PATTERN;
    using namespace ptx;
    extern __shared__ __align__(1024) unsigned char sm[];
    __shared__ __align__(8) uint64_t bars[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int fault_s;
    const uint32_t base = smem_u32(sm);
    const int warp = threadIdx.x >> 5;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0;
    const uint32_t sa = base, sb = base + 32768;              // A: 128 rows x 128 K; B: up to 256 rows x 128 K (or V: 128 keys x N)
    for (uint32_t i = threadIdx.x; i < (32768u + 65536u) / 4; i += 128) {
        uint32_t x = (i + 1u) * 2654435761u + blockIdx.x * 40503u;
        x ^= x >> 15; x *= 2246822519u; x ^= x >> 13;
        const uint32_t lo = 0x3c00u | (x & 0x83ffu), hi = 0x3c00u | ((x >> 16) & 0x83ffu);   // finite, |v| in [2^-7, 2)
        reinterpret_cast<uint32_t*>(sm)[i] = lo | (hi << 16);
    }
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars[0]), 1);
        mbar_init(smem_u32(&bars[1]), 1);
        fence_mbar_init();
        fault_s = 0;
    }
    if (warp == 0) {
        if (PAIR) { tmem_alloc_pair(smem_u32(&tmem_base_s), 512); tmem_relinquish_pair(); }
        else { tmem_alloc(smem_u32(&tmem_base_s), 512); tmem_relinquish(); }
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    constexpr uint32_t COL_P = 448;                             // the A operand of the TS form: 64 columns of packed bf16 pairs
    if (ts || pattern >= 2) {
        uint32_t r[32];
        for (int c = 0; c < 32; ++c) r[c] = 0x3c003c00u + (uint32_t)(c * 65537u + threadIdx.x);
        tmem_st32(tmem + ((uint32_t)(warp * 32) << 16) + COL_P, r);
        tmem_st32(tmem + ((uint32_t)(warp * 32) << 16) + COL_P + 32, r);
        tmem_wait_st();
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();
    tc_fence_after();
    if (rank == 0 && warp == 0) {
        if (elect_one()) {
            const uint32_t M = PAIR ? 256 : 128;
            const uint32_t idesc_ss = idesc_bf16(M, N, 0, 0), idesc_ts = idesc_bf16(M, N, 0, 1);
            const uint32_t bsub = (PAIR ? N / 2 : N) * 128;      // bytes of a 64-column sub-tile of the K-major B operand
            const uint32_t vlbo = 128 * 128;                      // MN-major B: 64-column groups 16 KB apart
            // descriptors once, so that the loop below is nothing but the MMAs
            uint64_t adesc[8], bdesc[8], vdesc[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                adesc[k] = smem_desc_sw128(sa + (k / 4) * 16384 + (k % 4) * 32, 16, 1024);
                bdesc[k] = smem_desc_sw128(sb + (k / 4) * bsub + (k % 4) * 32, 16, 1024);
                vdesc[k] = smem_desc_sw128(sb + k * 2048, vlbo, 1024);
            }
            auto ss = [&](uint32_t d, int k, bool acc) {
                if (PAIR) umma_ss_pair(d, adesc[k], bdesc[k], idesc_ss, acc); else umma_ss(d, adesc[k], bdesc[k], idesc_ss, acc);
            };
            auto tsf = [&](uint32_t d, int k, bool acc) {
                if (PAIR) umma_ts_pair(d, tmem + COL_P + k * 8, vdesc[k], idesc_ts, acc); else umma_ts(d, tmem + COL_P + k * 8, vdesc[k], idesc_ts, acc);
            };
            auto wait_round = [&](int r) -> bool {                // the commit of round r has arrived (bounded)
                const uint64_t w0 = globaltimer_ns();
                while (!mbar_try_wait(smem_u32(&bars[r & 1]), (uint32_t)((r >> 1) & 1)))
                    if (globaltimer_ns() - w0 > 1000000000ull) return false;
                return true;
            };
            const unsigned long long c0 = clock64(), t0 = globaltimer_ns();
            bool ok = true;
            for (int r = 0; r < rounds && ok; ++r) {
                const int b = r & 1;
                if (r >= 2 && !wait_round(r - 2)) { ok = false; break; }
                if (pattern == 0) {
                    const uint32_t d = tmem + (uint32_t)b * (uint32_t)N;
#pragma unroll
                    for (int k = 0; k < 8; ++k) { if (ts) tsf(d, k, k > 0); else ss(d, k, k > 0); }
                } else {
                    // two chains per round; with P in the way (patterns 2, 3 at N = 128) both rounds share one pair of accumulators
                    const uint32_t d0 = tmem + ((pattern >= 2 && 4 * N > (int)COL_P) ? 0u : (uint32_t)b * 2u * (uint32_t)N), d1 = d0 + (uint32_t)N;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int which = pattern == 3 ? i / 8 : i & 1, k = pattern == 3 ? i % 8 : i / 2;
                        if (which == 1 && pattern >= 2) tsf(d1, k, k > 0);
                        else ss(which ? d1 : d0, k, k > 0);
                    }
                }
                if (PAIR) umma_commit_pair(smem_u32(&bars[b])); else umma_commit(smem_u32(&bars[b]));
            }
            for (int r = rounds - 2; r < rounds && ok; ++r)
                if (r >= 0 && !wait_round(r)) ok = false;
            const unsigned long long c1 = clock64(), t1 = globaltimer_ns();
            if (!ok) fault_s = 1;
            if (blockIdx.x == 0) { res[0] = c1 - c0; res[1] = t1 - t0; }
            if (!ok) res[2] = 1;
        }
        __syncwarp();
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();
    if (fault_s) { const uint64_t w0 = globaltimer_ns(); while (globaltimer_ns() - w0 < 20000ull) { } }
    if (warp == 0) { if (PAIR) tmem_dealloc_pair(tmem, 512); else tmem_dealloc(tmem, 512); }
}

static int run_mma_rate(int pair, int N, int ts, int pattern, int rounds, unsigned long long* res, cudaStream_t st) {
    int rc, dev = 0, sms = 0;
    if ((rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice"))) return rc;
    if ((rc = check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "cudaDeviceGetAttribute"))) return rc;
    const size_t smem = 32768 + 65536;
    if ((rc = check_cuda(cudaMemsetAsync(res, 0, 3 * sizeof(unsigned long long), st), "cudaMemsetAsync(mma rate)"))) return rc;
    auto launch = [&](auto kern) -> int {
        int r2 = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem), "cudaFuncSetAttribute(mma rate)");
        if (r2) return r2;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(pair ? (unsigned)(sms / 2) * 2 : (unsigned)sms); cfg.blockDim = dim3(128); cfg.dynamicSmemBytes = smem; cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = pair ? 2 : 1; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        return check_cuda(cudaLaunchKernelEx(&cfg, kern, N, rounds, res), "mma rate launch");
    };
    if (pair) {
        switch (pattern) {
            case 0: rc = ts ? launch(mma_rate_kernel<1, 1, 0>) : launch(mma_rate_kernel<1, 0, 0>); break;
            case 1: rc = launch(mma_rate_kernel<1, 0, 1>); break;
            case 2: rc = launch(mma_rate_kernel<1, 0, 2>); break;
            default: rc = launch(mma_rate_kernel<1, 0, 3>); break;
        }
    } else {
        switch (pattern) {
            case 0: rc = ts ? launch(mma_rate_kernel<0, 1, 0>) : launch(mma_rate_kernel<0, 0, 0>); break;
            case 1: rc = launch(mma_rate_kernel<0, 0, 1>); break;
            case 2: rc = launch(mma_rate_kernel<0, 0, 2>); break;
            default: rc = launch(mma_rate_kernel<0, 0, 3>); break;
        }
    }
    if (rc) return rc;
    return check_cuda(cudaGetLastError(), "mma rate launch");
}

}  // namespace focus

extern "C" int focus_selftest_umma(int32_t D, const void* a, const void* b, const void* p, const void* v, float* s_out,
                                   float* o_out, int32_t* dev_status, void* stream) {
    using namespace focus;
    if (!a || !b || !p || !v || !s_out || !o_out || !dev_status) return fail(FOCUS_ERR_INVALID_ARG, "NULL argument");
    int rc = require_sm100();
    if (rc) return rc;
    switch (D) {
        case 64: return run_selftest<64>(a, b, p, v, s_out, o_out, dev_status, (cudaStream_t)stream);
        case 128: return run_selftest<128>(a, b, p, v, s_out, o_out, dev_status, (cudaStream_t)stream);
        case 256: return run_selftest<256>(a, b, p, v, s_out, o_out, dev_status, (cudaStream_t)stream);
    }
    return fail(FOCUS_ERR_UNSUPPORTED, "D (%d) must be 64, 128 or 256", D);
}

extern "C" int focus_selftest_umma_pair(const void* a, const void* b, const void* p, const void* v, float* s_out, float* o_out,
                                        int32_t* dev_status, void* stream) {
    using namespace focus;
    if (!a || !b || !p || !v || !s_out || !o_out || !dev_status) return fail(FOCUS_ERR_INVALID_ARG, "NULL argument");
    int rc = require_sm100();
    if (rc) return rc;
    return run_pair_selftest(a, b, p, v, s_out, o_out, dev_status, (cudaStream_t)stream);
}

extern "C" int focus_selftest_mma_rate(int32_t pair, int32_t N, int32_t ts, int32_t pattern, int32_t rounds,
                                       unsigned long long* result, void* stream) {
    using namespace focus;
    if (!result) return fail(FOCUS_ERR_INVALID_ARG, "result is NULL");
    if (pair < 0 || pair > 1 || ts < 0 || ts > 1 || pattern < 0 || pattern > 3 || rounds < 2 || rounds > 1000000)
        return fail(FOCUS_ERR_INVALID_ARG, "pair, ts in {0, 1}, pattern in 0..3, rounds in 2..1000000");
    if (N != 64 && N != 96 && N != 128 && N != 256) return fail(FOCUS_ERR_INVALID_ARG, "N must be 64, 96, 128 or 256");
    // tensor memory: two (pattern 0) or four accumulators of N columns, plus 64 columns of P for the TS form
    if ((ts || pattern >= 2) && N > 128) return fail(FOCUS_ERR_INVALID_ARG, "the TS form takes N <= 128 here");
    if (pattern == 1 && N > 128) return fail(FOCUS_ERR_INVALID_ARG, "two interleaved chains per commit take N <= 128 here");
    if (pattern >= 1 && ts) return fail(FOCUS_ERR_INVALID_ARG, "patterns 1-3 fix the forms of their chains: pass ts = 0");
    if (pair && N < 128) return fail(FOCUS_ERR_INVALID_ARG, "the CTA-pair form takes N = 128 or 256 here");
    int rc = require_sm100();
    if (rc) return rc;
    return run_mma_rate(pair, N, ts, pattern, rounds, result, (cudaStream_t)stream);
}
