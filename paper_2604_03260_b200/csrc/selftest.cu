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
