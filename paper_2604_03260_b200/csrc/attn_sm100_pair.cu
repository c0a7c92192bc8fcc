// focus_attn_fwd at head dimension 128 on pairs of CTAs (paper Sec. 2 and Appendix C, first equation).
//
// Two CTAs on neighbouring SMs (a cluster of two) share every tensor-core instruction: tcgen05.mma with
// cta_group::2 and M = 256, 128 rows per CTA.  An item is a head and two adjacent blocks of 256 queries, one block
// per CTA; the pair walks the union of the key tiles of its two blocks in lock-step.  Per key tile each CTA stages
// only HALF of K (64 of the 128 keys, all dimensions) and half of V (all keys, 64 of the 128 dimensions) in its own
// shared memory -- the MMA takes the two halves of its B operand from the two CTAs -- so the shared-memory traffic
// per key tile falls from 256 KB to 160 KB per SM and the ring holds twice as many tiles.  With one CTA per SM that
// traffic is level with the tensor pipe and the special-function unit and the three contend.
//
// Roles per CTA (384 threads):
//   warp 0        TMA producer: its block's two query tiles once per item, then its halves of K and V of every
//                 visited key tile.  Plain copies into its own shared memory (no multicast); their byte counts
//                 complete on the LEADER's mbarriers (the even CTA), which expect the bytes of both CTAs.
//   warp 1        leader: issues every MMA of the pair and signals completion to one mbarrier per CTA (two commits,
//                 no multicast).  Other CTA: idle apart from tensor-memory allocation.
//   warps 4-7     softmax for the block's query tile 0: S from its own tensor memory, mask, online max / sum,
//                 P (bf16) back to tensor memory, one arrival per warp on the leader's mbarrier
//   warps 8-11    softmax for query tile 1
// Each CTA writes the O rows and logsumexps of its own block.
//
// Every wait is bounded; a role that gives up raises the abort flag of both CTAs, every role then falls through to
// the common exit (cluster barrier, tensor-memory release) and dev_status says where it happened.
#include "attn_common.cuh"
#include "tma_host.cuh"

namespace focus {

template <int D>
struct PairCfg {
    static_assert(D == 128, "the CTA-pair kernel is written for head dimension 128");
    static constexpr uint32_t Q_SUB = 128 * 64 * 2;          // 128 queries x 64 dimensions
    static constexpr uint32_t Q_TILE = Q_SUB * (D / 64);
    static constexpr uint32_t K_SUB = 64 * 64 * 2;           // this CTA's 64 keys x 64 dimensions
    static constexpr uint32_t K_HALF = K_SUB * (D / 64);
    static constexpr uint32_t V_HALF = 128 * 64 * 2;         // 128 keys x this CTA's 64 dimensions
    static constexpr uint32_t STAGE = 16384;
    static_assert(K_HALF == STAGE && V_HALF == STAGE, "a ring stage holds one half tile");
    static constexpr int NSTAGE = 8;
    static constexpr uint32_t SMEM_BYTES = 1024 + 2 * Q_TILE + NSTAGE * STAGE;
    static constexpr uint32_t COL_S0 = 0, COL_S1 = 128, COL_O0 = 256, COL_O1 = 256 + D;
    static constexpr int THREADS = 384;
};

struct PairCtl {
    uint64_t q_full, q_empty;             // q_full, p_full, kv_full are waited on in the leader only
    uint64_t s_full[2], p_full[2], o_full[2];
    uint64_t kv_full[8], kv_empty[8];
    uint64_t drain;
    uint32_t tmem_base;
    int abort_flag;
};

// bounded wait on a local mbarrier; gives up early when a role of either CTA has given up
template <bool CLUSTER_ACQUIRE = false>
__device__ __forceinline__ bool pair_wait(uint64_t* bar, uint32_t parity, PairCtl* ctl) {
    const uint32_t a = smem_u32(bar);
    auto try_once = [&]() { return CLUSTER_ACQUIRE ? mbar_try_wait_cluster(a, parity) : mbar_try_wait(a, parity); };
    if (try_once()) return true;
    const uint64_t t0 = globaltimer_ns();
    for (;;) {
#pragma unroll 1
        for (int it = 0; it < 128; ++it)
            if (try_once()) return true;
        if (*(volatile int*)&ctl->abort_flag) return false;
        if (globaltimer_ns() - t0 > 4000000000ull) return false;
    }
}

__device__ __forceinline__ void pair_report_timeout(const AttnParams& p, PairCtl* ctl, uint32_t peer, int where, int item) {
    *(volatile int*)&ctl->abort_flag = 1;
    st_shared_cluster_u32(mapa_shared(smem_u32(&ctl->abort_flag), peer), 1u);
    if (p.status && atomicCAS(p.status, 0, 1) == 0) {
        p.status[1] = where;
        p.status[2] = item;
        p.status[3] = (int)blockIdx.x;
    }
}

template <int D, bool SOFTCAP>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PairCfg<D>::THREADS, 1)
focus_attn_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, const AttnParams p) {
    using C = PairCfg<D>;
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) PairCtl ctl;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sq = base;                                 // this CTA's two query tiles
    const uint32_t skv = base + 2 * C::Q_TILE;                 // ring of half tiles of K / V
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank(), peer = rank ^ 1u;
    const bool leader = rank == 0;
    const int npairs = (int)cluster_count_x(), pair_id = (int)cluster_id_x();

    if (p.sorted && __ldg(p.counters + 4) != 0ull) {      // more mask values than the sorted layout holds: refuse (both CTAs alike)
        if (threadIdx.x == 0 && p.status && atomicCAS(p.status, 0, 2) == 0) {
            p.status[1] = 1; p.status[2] = 0; p.status[3] = (int)blockIdx.x;
        }
        return;
    }
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&ctl.q_full), 1);
        mbar_init(smem_u32(&ctl.q_empty), 1);
        mbar_init(smem_u32(&ctl.drain), 1);
        for (int x = 0; x < 2; ++x) {
            mbar_init(smem_u32(&ctl.s_full[x]), 1);
            mbar_init(smem_u32(&ctl.p_full[x]), 8);            // one arrival per softmax warp of the tile, both CTAs
            mbar_init(smem_u32(&ctl.o_full[x]), 1);
        }
        for (int s = 0; s < C::NSTAGE; ++s) {
            mbar_init(smem_u32(&ctl.kv_full[s]), 1);
            mbar_init(smem_u32(&ctl.kv_empty[s]), 1);
        }
        ctl.abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(&ctl.tmem_base), 512);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                 // the other CTA's mbarriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem = ctl.tmem_base;

    if (warp < 4) reg_dec<REGS_CONTROL>();
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            prefetch_tmap(&tm_q); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v);
            const uint32_t lead_q_full = mapa_shared(smem_u32(&ctl.q_full), 0);
            long long nload = 0;
            int it = 0;
            bool ok = true;
            Item t;
            for (int round = 0; ok && item_of(p, round, t, npairs, pair_id); ++round) {
                const int hq = t.hq, b = t.bb, h = t.h, hk = h / p.G;
                const int A = 2 * t.A + (int)rank;                    // this CTA's block of 256 queries
                const long long item = t.id;
                TileWalk walk;
                walk.init(p, hq, t.A * 4, 4);
                int kb = walk.next();
                if (kb < 0) continue;
                if (it > 0 && !pair_wait(&ctl.q_empty, (it - 1) & 1, &ctl)) { pair_report_timeout(p, &ctl, peer, 10, (int)item); break; }
                if (leader) mbar_arrive_expect_tx(smem_u32(&ctl.q_full), 4 * C::Q_TILE);     // two tiles from each CTA
                const int qh = p.sorted ? hq : h, qb = p.sorted ? 0 : b;
                const int kh = p.sorted ? b * p.Hkv + hk : hk;
                for (int x = 0; x < 2; ++x)
                    for (int c = 0; c < D / 64; ++c)
                        tma_load_4d_pair(sq + x * C::Q_TILE + c * C::Q_SUB, &tm_q, lead_q_full, c * 64, (A * 2 + x) * 128, qh, qb);
                // this CTA's half of one K or V tile into the next stage of the ring
                auto load_half = [&](bool is_v, int tile) {
                    const int slot = (int)(nload % C::NSTAGE);
                    const long long use = nload / C::NSTAGE;
                    if (use > 0 && !pair_wait(&ctl.kv_empty[slot], (uint32_t)((use - 1) & 1), &ctl)) {
                        pair_report_timeout(p, &ctl, peer, 11, (int)item);
                        ok = false;
                        return;
                    }
                    if (leader) mbar_arrive_expect_tx(smem_u32(&ctl.kv_full[slot]), 2 * C::STAGE);
                    const uint32_t bar = mapa_shared(smem_u32(&ctl.kv_full[slot]), 0);
                    const uint32_t dst = skv + slot * C::STAGE;
                    if (is_v) {         // all 128 keys x its 64 dimensions
                        tma_load_4d_pair(dst, &tm_v, bar, (int)rank * 64, tile * 128, kh, qb);
                    } else {            // its 64 keys x all dimensions
                        for (int c = 0; c < D / 64; ++c)
                            tma_load_4d_pair(dst + c * C::K_SUB, &tm_k, bar, c * 64, tile * 128 + (int)rank * 64, kh, qb);
                    }
                    ++nload;
                };
                for (; ok && kb >= 0; kb = walk.next()) {
                    load_half(false, kb);
                    if (ok) load_half(true, kb);
                }
                ++it;
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (leader) {
            constexpr uint32_t IDESC_S = idesc_bf16(256, 128, 0, 0);
            constexpr uint32_t IDESC_O = idesc_bf16(256, D, 0, 1);
            long long nuse = 0;
            uint32_t np[2] = {0, 0};
            int it = 0;
            bool ok = true;
            const uint64_t qdesc0 = smem_desc_sw128(sq, 16, 1024);
            const uint64_t kdesc0 = smem_desc_sw128(skv, 16, 1024);                 // K halves: K-major, 64 rows
            const uint64_t vdesc0 = smem_desc_sw128(skv, C::V_HALF, 1024);           // V halves: MN-major, one 64-column chunk
            // the same mbarrier in this CTA and in the other one
            auto commit_both = [&](uint64_t* bar) {
                if (elect_one()) {
                    const uint32_t a = smem_u32(bar);
                    umma_commit_pair(a);
                    umma_commit_pair(mapa_shared(a, 1));
                }
            };
            auto issue_s = [&](int x, int kslot) {
                if (elect_one()) {
                    const uint32_t d = tmem + (x ? C::COL_S1 : C::COL_S0);
                    const uint64_t ad = qdesc0 + (uint64_t)((x * C::Q_TILE) >> 4);
                    const uint64_t bd = kdesc0 + (uint64_t)((kslot * C::STAGE) >> 4);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks)
                        umma_ss_pair(d, ad + (uint64_t)(((ks / 4) * C::Q_SUB + (ks % 4) * 32) >> 4),
                                     bd + (uint64_t)(((ks / 4) * C::K_SUB + (ks % 4) * 32) >> 4), IDESC_S, ks > 0);
                }
            };
            auto issue_o = [&](int x, int vslot, bool first) {
                if (elect_one()) {
                    const uint32_t d = tmem + (x ? C::COL_O1 : C::COL_O0);
                    const uint32_t a = tmem + (x ? C::COL_S1 : C::COL_S0);
                    const uint64_t bd = vdesc0 + (uint64_t)((vslot * C::STAGE) >> 4);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        umma_ts_pair(d, a + ks * 8, bd + (uint64_t)((ks * 2048) >> 4), IDESC_O, (!first) || ks > 0);
                }
            };
            auto wait_kv = [&](int& slot, int where, int item) -> bool {
                slot = (int)(nuse % C::NSTAGE);
                if (!pair_wait<true>(&ctl.kv_full[slot], (uint32_t)((nuse / C::NSTAGE) & 1), &ctl)) {
                    pair_report_timeout(p, &ctl, peer, where, item);
                    return false;
                }
                ++nuse;
                return true;
            };
            Item t;
            for (int round = 0; ok && item_of(p, round, t, npairs, pair_id); ++round) {
                const long long item = t.id;
                TileWalk walk;
                walk.init(p, t.hq, t.A * 4, 4);
                int cur = walk.next();
                if (cur < 0) continue;
                if (!pair_wait<true>(&ctl.q_full, it & 1, &ctl)) { pair_report_timeout(p, &ctl, peer, 20, (int)item); break; }
                {
                    int slot;
                    if (!wait_kv(slot, 21, (int)item)) break;
                    tc_fence_after();
                    issue_s(0, slot); commit_both(&ctl.s_full[0]);
                    issue_s(1, slot); commit_both(&ctl.s_full[1]);
                    commit_both(&ctl.kv_empty[slot]);
                }
                bool first = true;
                while (cur >= 0) {
                    const int nxt = walk.next();
                    int vslot = 0, kslot = 0;
                    if (!wait_kv(vslot, 22, (int)item)) { ok = false; break; }
                    if (nxt >= 0 && !wait_kv(kslot, 23, (int)item)) { ok = false; break; }
                    if (nxt < 0) commit_both(&ctl.q_empty);     // every S of this item has been issued
                    // query tile 0 of both blocks
                    if (!pair_wait<true>(&ctl.p_full[0], np[0] & 1, &ctl)) { pair_report_timeout(p, &ctl, peer, 24, (int)item); ok = false; break; }
                    ++np[0];
                    tc_fence_after();
                    issue_o(0, vslot, first);
                    if (nxt >= 0) { issue_s(0, kslot); commit_both(&ctl.s_full[0]); }
                    else commit_both(&ctl.o_full[0]);
                    // query tile 1 of both blocks
                    if (!pair_wait<true>(&ctl.p_full[1], np[1] & 1, &ctl)) { pair_report_timeout(p, &ctl, peer, 25, (int)item); ok = false; break; }
                    ++np[1];
                    tc_fence_after();
                    issue_o(1, vslot, first);
                    commit_both(&ctl.kv_empty[vslot]);
                    if (nxt >= 0) {
                        issue_s(1, kslot); commit_both(&ctl.s_full[1]);
                        commit_both(&ctl.kv_empty[kslot]);
                    } else {
                        commit_both(&ctl.o_full[1]);
                    }
                    first = false;
                    cur = nxt;
                }
                ++it;
            }
            // nothing of the pair's tensor-core work may be in flight when the CTAs leave
            if (elect_one()) umma_commit_pair(smem_u32(&ctl.drain));
            pair_wait(&ctl.drain, 0, &ctl);
        }
        __syncwarp();
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ softmax + epilogue (both CTAs)
        reg_inc<REGS_SOFTMAX_2WG>();
        const int x = (warp - 4) >> 2;                       // query tile of this warpgroup
        const int row_in_tile = ((warp & 3) << 5) | lane;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_o = tmem + lane_base + (x ? C::COL_O1 : C::COL_O0);
        const uint32_t t_s = tmem + lane_base + (x ? C::COL_S1 : C::COL_S0);
        const uint32_t lead_p_full = mapa_shared(smem_u32(&ctl.p_full[x]), 0);
        const float sl2 = SOFTCAP ? p.softcap * LOG2E : p.scale * LOG2E;
        const float cap_in = SOFTCAP ? p.scale / p.softcap : 0.f;
        uint32_t ns = 0;
        int it = 0;
        bool ok = true;
        Item t;
        for (int round = 0; ok && item_of(p, round, t, npairs, pair_id); ++round) {
            const int hq = t.hq, bb = t.bb, h = t.h;
            const long long item = t.id;
            const int hk = bb * p.Hkv + h / p.G;
            const int A = 2 * t.A + (int)rank;
            const int a = A * 2 + x;
            TileWalk walk;
            walk.init(p, hq, t.A * 4, 4);
            int kb = walk.next();
            if (kb < 0) continue;
            long long i = (long long)a * 128 + row_in_tile;
            int wmin = 0, wmax = 0;
            if (p.sorted) {
                i = A < p.nqblk ? __ldg(p.perm_q + (size_t)hq * p.nqp + i) : -1;     // -1: padding, or no second block
                wmin = __reduce_min_sync(0xffffffffu, i < 0 ? 0x7fffffff : (int)i);
                wmax = __reduce_max_sync(0xffffffffu, (int)i);
            }
            const bool valid = i >= 0 && i < p.n;
            const uint32_t mi = (valid && !p.dense) ? __ldg(p.mq + (size_t)hq * p.n + i) : 0u;
            const uint32_t aq = (!p.dense && !p.sorted && a < p.nqt) ? __ldg(p.andq + (size_t)hq * p.nqt + a) : 0u;
            const long long dfar = (long long)a * 128 - p.w;
            const int f_x = (!p.dense && dfar > 0) ? (int)(dfar / 128) : 0;
            float m_used = -INFINITY, l = 0.f;
            bool first = true;
            for (; kb >= 0; kb = walk.next()) {
                TileMask tm;
                if (p.sorted) {
                    const bool share = (mi & __ldg(p.cls_k + (size_t)hk * FOCUS_MAX_CLASSES + walk.jk)) != 0u;
                    build_tile_mask_sorted(tm, p.w, p.perm_k + (size_t)hk * p.nkp + (size_t)kb * 128, share,
                                           valid ? (int)i : -1, wmin, wmax);
                } else {
                    build_tile_mask(tm, p, a, kb, i, mi, aq, f_x, hk);
                }
                if (!pair_wait(&ctl.s_full[x], ns & 1, &ctl)) { pair_report_timeout(p, &ctl, peer, 30 + x, (int)item); ok = false; break; }
                tc_fence_after();
                uint32_t pk[64];
                if (tm.all_masked) {
#pragma unroll
                    for (int c = 0; c < 64; ++c) pk[c] = 0u;
                } else {
                    uint32_t sr[128];
#pragma unroll
                    for (int c = 0; c < 4; ++c) tmem_ld32(t_s + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[c * 32]));
                    tmem_wait_ld();
                    if (SOFTCAP) {
#pragma unroll
                        for (int c = 0; c < 128; ++c) sr[c] = __float_as_uint(tanh_approx(__uint_as_float(sr[c]) * cap_in));
                    }
                    if (tm.masked) {
#pragma unroll
                        for (int c = 0; c < 128; ++c) sr[c] = ((tm.kw[c >> 5] >> (c & 31)) & 1u) ? sr[c] : 0xff800000u;      // -inf
                    }
                    float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                    for (int c = 0; c < 128; c += 8) {
                        mx0 = max3(mx0, __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]));
                        mx1 = max3(mx1, __uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3]));
                        mx2 = max3(mx2, __uint_as_float(sr[c + 4]), __uint_as_float(sr[c + 5]));
                        mx3 = max3(mx3, __uint_as_float(sr[c + 6]), __uint_as_float(sr[c + 7]));
                    }
                    const float mt = max3(mx0, mx1, fmaxf(mx2, mx3)) * sl2;      // log2 units (sl2 > 0; -inf stays -inf)
                    // lazy maximum: raise the reference only when it lags by more than the threshold
                    float factor = 1.f;
                    bool raise = false;
                    if (m_used == -INFINITY) {
                        m_used = mt;
                    } else if (mt > m_used + RESCALE_THRESHOLD) {
                        factor = ex2_approx(m_used - mt);
                        m_used = mt;
                        raise = true;
                    }
                    if (__any_sync(0xffffffffu, raise) && !first) {
                        // the previous P V of this query tile has completed: its commit precedes s_full
#pragma unroll 1
                        for (int c = 0; c < D / 16; ++c) {
                            uint32_t ov[16];
                            tmem_ld16(t_o + c * 16, ov);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < 16; ++e) ov[e] = __float_as_uint(__uint_as_float(ov[e]) * factor);
                            tmem_st16(t_o + c * 16, ov);
                        }
                    }
                    l *= factor;
                    const float msub = m_used == -INFINITY ? 0.f : m_used;
                    const float2 sl2v = make_float2(sl2, sl2), nmv = make_float2(-msub, -msub);
                    float2 acc[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[e] = make_float2(0.f, 0.f);
#pragma unroll
                    for (int c = 0; c < 128; c += 8) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float2 xv = __ffma2_rn(make_float2(__uint_as_float(sr[c + 2 * e]),
                                                                     __uint_as_float(sr[c + 2 * e + 1])), sl2v, nmv);
                            float2 pr;
                            pr.x = ex2_approx(xv.x);
                            pr.y = ex2_approx(xv.y);
                            acc[e] = __fadd2_rn(acc[e], pr);
                            pk[(c >> 1) + e] = pack_bf16x2(pr.x, pr.y);
                        }
                    }
                    l += (acc[0].x + acc[0].y) + (acc[1].x + acc[1].y) + ((acc[2].x + acc[2].y) + (acc[3].x + acc[3].y));
                }
#pragma unroll
                for (int c = 0; c < 2; ++c) tmem_st32(t_s + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&pk[c * 32]));
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(lead_p_full);
                ++ns;
                first = false;
            }
            if (!ok) break;
            // ---- epilogue: O / l -> bf16 -> global, lse
            if (!pair_wait(&ctl.o_full[x], it & 1, &ctl)) { pair_report_timeout(p, &ctl, peer, 40 + x, (int)item); break; }
            tc_fence_after();
            const float inv_l = l > 0.f ? 1.f / l : 0.f;        // a row without any pair (possible in a partial pass): zeros, lse = -inf
            __nv_bfloat16* orow = p.o + (size_t)bb * p.o_sb + (size_t)h * p.o_sh + (size_t)(valid ? i : 0) * p.o_sn;
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
                uint32_t ov[32];
                tmem_ld32(t_o + c * 32, ov);
                tmem_wait_ld();
                if (valid && p.o32) {
                    float* o32row = p.o32 + ((size_t)hq * p.n + (size_t)i) * D + c * 32;
#pragma unroll
                    for (int e = 0; e < 32; e += 4)
                        *reinterpret_cast<float4*>(o32row + e) =
                            make_float4(__uint_as_float(ov[e]) * inv_l, __uint_as_float(ov[e + 1]) * inv_l,
                                        __uint_as_float(ov[e + 2]) * inv_l, __uint_as_float(ov[e + 3]) * inv_l);
                } else if (valid) {
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint4 w4;
                        w4.x = pack_bf16x2(__uint_as_float(ov[e]) * inv_l, __uint_as_float(ov[e + 1]) * inv_l);
                        w4.y = pack_bf16x2(__uint_as_float(ov[e + 2]) * inv_l, __uint_as_float(ov[e + 3]) * inv_l);
                        w4.z = pack_bf16x2(__uint_as_float(ov[e + 4]) * inv_l, __uint_as_float(ov[e + 5]) * inv_l);
                        w4.w = pack_bf16x2(__uint_as_float(ov[e + 6]) * inv_l, __uint_as_float(ov[e + 7]) * inv_l);
                        *reinterpret_cast<uint4*>(orow + c * 32 + e) = w4;
                    }
                }
            }
            if (valid) p.lse[(size_t)hq * p.n + i] = (m_used + lg2_approx(l)) * LN2;
            tc_fence_before();
            ++it;
        }
    }
    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*(volatile int*)&ctl.abort_flag) {
        // a role gave up: let copies that were already issued land before either CTA leaves
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 100000ull) { }
    }
    cluster_sync_all();                 // neither CTA leaves, or frees tensor memory, while the other may still use it
    if (warp == 1) tmem_dealloc_pair(tmem, 512);
}

template <bool SOFTCAP>
static int launch_pair_t(const AttnArgs& a, cudaStream_t st) {
    constexpr int D = 128;
    using C = PairCfg<D>;
    CUtensorMap tq, tk, tv;
    int rc;
    const bool sorted = a.ws && !a.local_pass &&
                        (a.L.layout == FOCUS_LAYOUT_CLASS_SORTED || a.L.layout == FOCUS_LAYOUT_SORTED_LOCAL);
    if (sorted) {
        char* ws = const_cast<char*>(a.ws);
        if ((rc = launch_gather_sorted(&a.s, a.q, a.s.Hq, true, a.L, a.ws, ws + a.L.qs, st))) return rc;
        if ((rc = launch_gather_sorted(&a.s, a.k, a.s.Hkv, false, a.L, a.ws, ws + a.L.ks, st))) return rc;
        if ((rc = launch_gather_sorted(&a.s, a.v, a.s.Hkv, false, a.L, a.ws, ws + a.L.vs, st))) return rc;
        const int HQ = a.s.batch * a.s.Hq, HK = a.s.batch * a.s.Hkv;
        const focus_tensor sq_t{ws + a.L.qs, (int64_t)HQ * a.L.nqp * D, (int64_t)a.L.nqp * D, D};
        const focus_tensor sk_t{ws + a.L.ks, (int64_t)HK * a.L.nkp * D, (int64_t)a.L.nkp * D, D};
        const focus_tensor sv_t{ws + a.L.vs, (int64_t)HK * a.L.nkp * D, (int64_t)a.L.nkp * D, D};
        if ((rc = make_tmap_qkv(&tq, sq_t, 1, HQ, a.L.nqp, D))) return rc;
        if ((rc = make_tmap_qkv(&tk, sk_t, 1, HK, a.L.nkp, D, 64))) return rc;
        if ((rc = make_tmap_qkv(&tv, sv_t, 1, HK, a.L.nkp, D))) return rc;
    } else {
        if ((rc = make_tmap_qkv(&tq, a.q, a.s.batch, a.s.Hq, a.s.n, D))) return rc;
        if ((rc = make_tmap_qkv(&tk, a.k, a.s.batch, a.s.Hkv, a.s.n, D, 64))) return rc;
        if ((rc = make_tmap_qkv(&tv, a.v, a.s.batch, a.s.Hkv, a.s.n, D))) return rc;
    }
    AttnParams p;
    p.B = a.s.batch; p.Hq = a.s.Hq; p.Hkv = a.s.Hkv; p.G = a.s.Hq / a.s.Hkv; p.n = a.s.n; p.w = a.s.window; p.K = a.s.K;
    p.nqb = cdiv(cdiv(a.s.n, 256), 2);                       // items per head: pairs of 256-query blocks
    p.nqt = cdiv(a.s.n, 128); p.nkt = cdiv(a.s.n, 128); p.nkw = cdiv(p.nkt, 32);
    p.dense = a.ws ? 0 : 1;
    p.scale = a.scale; p.softcap = a.s.softcap;
    p.mq = a.mq;
    p.gbits = a.ws ? reinterpret_cast<const uint32_t*>(a.ws + a.L.gbits) : nullptr;
    p.live = a.ws ? reinterpret_cast<const uint32_t*>(a.ws + a.L.live) : nullptr;
    p.andq = a.ws ? reinterpret_cast<const uint32_t*>(a.ws + a.L.andq) : nullptr;
    p.andk = a.ws ? reinterpret_cast<const uint32_t*>(a.ws + a.L.andk) : nullptr;
    p.o = reinterpret_cast<__nv_bfloat16*>(a.o.ptr);
    p.o_sb = a.o.stride_b; p.o_sh = a.o.stride_h; p.o_sn = a.o.stride_n;
    p.lse = a.lse;
    p.status = a.dev_status;
    p.nitems = (long long)a.s.batch * a.s.Hq * p.nqb;
    p.sorted = sorted ? 1 : 0;
    p.nqp = a.L.nqp; p.nkp = a.L.nkp; p.nqblk = a.L.nqp / 256;
    p.ipb = 1;
    p.perm_q = sorted ? reinterpret_cast<const int32_t*>(a.ws + a.L.perm_q) : nullptr;
    p.perm_k = sorted ? reinterpret_cast<const int32_t*>(a.ws + a.L.perm_k) : nullptr;
    p.cls_k = sorted ? reinterpret_cast<const uint32_t*>(a.ws + a.L.cls_k) : nullptr;
    p.ncls_k = sorted ? reinterpret_cast<const int32_t*>(a.ws + a.L.ncls_k) : nullptr;
    p.qrange = sorted ? reinterpret_cast<const int32_t*>(a.ws + a.L.qrange) : nullptr;
    p.order = sorted ? reinterpret_cast<const int32_t*>(a.ws + a.L.order_pair) : nullptr;
    p.counters = a.ws ? reinterpret_cast<const unsigned long long*>(a.ws + a.L.counters) : nullptr;
    p.gate_g = nullptr; p.gate_ld = 0; p.gate_hl = 0.f;
    p.local_only = a.local_pass ? 1 : 0;
    p.o32 = a.o32;
    if (sorted) p.nitems = (long long)a.s.batch * a.s.Hq * cdiv(p.nqblk, 2);
    auto kern = focus_attn_pair_kernel<D, SOFTCAP>;
    if ((rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM_BYTES),
                         "cudaFuncSetAttribute(pair attention)")))
        return rc;
    // as many pairs as can be resident together (one CTA per SM), at most one per item
    int dev = 0, sms = 0;
    if ((rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice"))) return rc;
    if ((rc = check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "cudaDeviceGetAttribute"))) return rc;
    int pairs = sms / 2;
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(2 * pairs));
        cfg.blockDim = dim3(C::THREADS);
        cfg.dynamicSmemBytes = C::SMEM_BYTES;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int resident = 0;
        if (cudaOccupancyMaxActiveClusters(&resident, kern, &cfg) == cudaSuccess && resident > 0 && resident < pairs) pairs = resident;
        else (void)cudaGetLastError();
    }
    if (p.nitems < pairs) pairs = (int)p.nitems;
    kern<<<2 * pairs, C::THREADS, C::SMEM_BYTES, st>>>(tq, tk, tv, p);
    return check_cuda(cudaGetLastError(), "pair attention kernel launch");
}

int launch_attn_pair(const AttnArgs& a, cudaStream_t st) {
    return a.s.softcap > 0.f ? launch_pair_t<true>(a, st) : launch_pair_t<false>(a, st);
}

}  // namespace focus
