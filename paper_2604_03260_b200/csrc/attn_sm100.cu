// focus_attn_fwd for sm_100a: persistent, warp-specialised attention forward over the attended
// pairs of the Focus mask (paper Sec. 2 and Appendix D, first equation).
//
// One CTA per SM works through (head, 256-query block) items.  Per item, two 128-row query tiles
// share every key/value tile that is fetched:
//   warp 0        TMA producer: Q tiles once per item, then K and V tiles of every visited key tile
//                 into a ring of shared-memory stages (128-byte swizzle)
//   warp 1        MMA issuer: S_x = Q_x K^T and O_x += P_x V with tcgen05.mma, accumulators in TMEM
//                 (the whole warp runs the loop, one elected lane issues)
//   warps 4-7     softmax for query tile 0: tcgen05.ld S, mask, online max/sum, P (bf16) back to TMEM
//   warps 8-11    softmax for query tile 1
// After the split into roles the control warpgroup hands registers to the softmax warpgroups
// (setmaxnreg).  The two softmax groups alternate on the tensor pipe: while one computes exponentials
// the MMAs of the other run.  The running maximum is raised lazily (only when it grows by more than
// 2^8), and then the owner of the row rescales its O row in TMEM itself.
//
// Head dimension 256 does not leave room in TMEM for two query tiles (O alone is 256 columns), so
// there an item is a single 128-row query tile, S is double-buffered over consecutive key tiles
// and one warpgroup does the softmax while the MMAs of the neighbouring tiles run.
//
// Which key tiles are visited, and in which order of items:
//   dense mode      every tile up to the diagonal
//   original layout far tiles (every pair beyond the window) only when the live bitmap says the OR
//                   of the query-tile masks meets the OR of the key-tile masks; near tiles always
//   class-sorted    Q, K, V are the copies gathered into the class-sorted order; per key class the
//                   range of sorted key tiles listed for the query block; a row's kept columns of a
//                   tile are a contiguous range found from the tile's ascending positions; O and lse
//                   go straight to the rows' original positions
// Items are laid out KV head by KV head (class-sorted: most key tiles first inside a group) and
// dealt to the CTAs in alternating direction round by round.
#include "attn_common.cuh"
#include "tma_host.cuh"

namespace focus {

// GATE: 0 = no soft gate, else the number of 8-float chunks of a token's soft assignment (1, 2 or 4: K <= 8, 16, 32)
template <int D, int GATE = 0>
struct AttnCfg {
    static constexpr int NQ = (D == 256) ? 1 : 2;            // 128-row query tiles per item
    static constexpr int SUBT = D / 64;
    static constexpr uint32_t SUB_BYTES = 128 * 64 * 2;
    static constexpr uint32_t TILE_BYTES = SUB_BYTES * SUBT;
    // The K/V ring.  Up to D = 128 a stage holds a whole 128-key tile of K or of V.  At D = 256 only two such stages
    // would fit next to Q, so a tile travels as two half stages cut along the contraction dimension of its MMA (the
    // full-width MMA shapes stay): a K half is all 128 keys x 128 of the 256 head dimensions, a V half is 64 keys x
    // all 256 dimensions.  Five half stages fit, and a half goes back to the producer as soon as its own MMAs are done.
    static constexpr int PARTS = (D == 256) ? 2 : 1;         // ring stages per tile
    static constexpr uint32_t STAGE_BYTES = TILE_BYTES / PARTS;
    static constexpr int NSTAGE = (D == 256) ? (GATE ? 4 : 5) : ((D == 128) ? (GATE == 4 ? 3 : (GATE ? 4 : 5)) : 8);
    // soft gate: per softmax warpgroup two buffers of 128 key assignments, 8 GATE floats each (after the ring)
    static constexpr uint32_t GATE_ROW_BYTES = 32 * (GATE ? GATE : 1);
    static constexpr uint32_t GATE_BUF_BYTES = 128 * GATE_ROW_BYTES;
    static_assert(!(D == 256 && GATE == 4), "no room for the K/V ring beside 64 KB of gate buffers at D = 256");
    static constexpr uint32_t SMEM_BYTES = 1024 + NQ * TILE_BYTES + NSTAGE * STAGE_BYTES + (GATE ? 4 * GATE_BUF_BYTES : 0);
    // Ring order of the tiles.  With one query tile the S of the next key tile is issued before the current P V, so
    // K(next) travels ahead of V(current); with two query tiles V(current) is consumed and released first.
    static constexpr bool K_AHEAD = NQ == 1;
    static constexpr uint32_t COL_S0 = 0, COL_S1 = 128, COL_O0 = 256, COL_O1 = 256 + D;
    // With a single query tile two threads share a row: each of the two softmax warpgroups owns one 64-column
    // half of every key tile (its S columns, its P columns, its part of the row sum) and one half of the O row.
    static constexpr int NSPLIT = NQ == 1 ? 2 : 1;
    static constexpr int NC = 128 / NSPLIT;                  // S columns per softmax thread
    static constexpr int THREADS = 128 + 128 * NQ * NSPLIT;
};

struct SharedCtl {
    uint64_t q_full, q_empty;
    uint64_t s_full[2], p_full[2], o_full[2];
    uint64_t pv_done;
    uint64_t xchg[4];                 // split rows, per 32-row quadrant: both column halves have published a per-row value
    uint64_t gbar[2];                 // soft gate, per softmax warpgroup: the key assignments of the tile are in shared memory
    uint64_t kv_full[8], kv_empty[8];
    unsigned long long limit_ns;      // how long a wait may last before the role gives up
    uint32_t tmem_base;
    int abort_flag;
};

// bounded wait that also gives up when another role of the CTA has already given up
__device__ __forceinline__ bool ctl_wait(uint64_t* bar, uint32_t parity, SharedCtl* ctl) {
    const uint32_t a = smem_u32(bar);
    if (mbar_try_wait(a, parity)) return true;
    const uint64_t t0 = globaltimer_ns();
    for (;;) {
#pragma unroll 1
        for (int it = 0; it < 128; ++it)
            if (mbar_try_wait(a, parity)) return true;
        if (*(volatile int*)&ctl->abort_flag) return false;
        if (globaltimer_ns() - t0 > ctl->limit_ns) return false;
    }
}

__device__ __forceinline__ void report_timeout(const AttnParams& p, SharedCtl* ctl, int where, int item) {
    *(volatile int*)&ctl->abort_flag = 1;
    if (p.status && atomicCAS(p.status, 0, 1) == 0) {
        p.status[1] = where;
        p.status[2] = item;
        p.status[3] = (int)blockIdx.x;
    }
}

template <int D, bool SOFTCAP, int GATE>
__global__ void __launch_bounds__(AttnCfg<D, GATE>::THREADS, 1)
focus_attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const AttnParams p) {
    using C = AttnCfg<D, GATE>;
    constexpr int NQ = C::NQ;
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) SharedCtl ctl;
    // split rows: [parity][column half][row] row maxima, at the end row sums (the other instantiations have no room to spare)
    // (bf16: a rounded row maximum serves as well as the exact one as long as both threads use the same value)
    __shared__ __nv_bfloat16 xval_s[C::NSPLIT == 2 ? 2 * 2 * 128 : 1];
    auto xval = [&](int par, int hf, int row) -> __nv_bfloat16& { return xval_s[C::NSPLIT == 2 ? (par * 2 + hf) * 128 + row : 0]; };
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sq = base;                                 // NQ query tiles
    const uint32_t skv = base + NQ * C::TILE_BYTES;            // ring of K / V tiles
    unsigned char* const gate_sm = smem_raw + (base - smem_u32(smem_raw)) + NQ * C::TILE_BYTES + C::NSTAGE * C::STAGE_BYTES;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (p.sorted && __ldg(p.counters + 4) != 0ull) {      // more mask values than the sorted layout holds: refuse
        if (threadIdx.x == 0 && p.status && atomicCAS(p.status, 0, 2) == 0) {
            p.status[1] = 1; p.status[2] = 0; p.status[3] = (int)blockIdx.x;
        }
        return;
    }
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&ctl.q_full), 1);
        mbar_init(smem_u32(&ctl.q_empty), 1);
        mbar_init(smem_u32(&ctl.pv_done), 1);
        for (int qd = 0; qd < 4; ++qd) mbar_init(smem_u32(&ctl.xchg[qd]), 2);
        for (int g = 0; g < 2; ++g) mbar_init(smem_u32(&ctl.gbar[g]), 4);
        for (int x = 0; x < 2; ++x) {
            mbar_init(smem_u32(&ctl.s_full[x]), 1);
            mbar_init(smem_u32(&ctl.p_full[x]), 128 * C::NSPLIT);
            mbar_init(smem_u32(&ctl.o_full[x]), 1);
        }
        for (int s = 0; s < C::NSTAGE; ++s) {
            mbar_init(smem_u32(&ctl.kv_full[s]), 1);
            mbar_init(smem_u32(&ctl.kv_empty[s]), 1);
        }
        ctl.abort_flag = 0;
        ctl.limit_ns = p.wait_limit_ns;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl.tmem_base), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctl.tmem_base;

    if (warp < 4) reg_dec<REGS_CONTROL>();
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tmap(&tm_q); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v);
            long long nload = 0;
            int it = 0;                     // items processed (items without key tiles are skipped by every role)
            bool ok = true;
            Item t;
            for (int round = 0; ok && item_of(p, round, t, (int)gridDim.x, (int)blockIdx.x); ++round) {
                const int A = t.A, hq = t.hq, b = t.bb, h = t.h, hk = h / p.G;
                const long long item = t.id;
                TileWalk walk;
                walk.init(p, hq, A * NQ, NQ);
                int kb = walk.next();
                if (kb < 0) continue;
                if (it > 0 && !ctl_wait(&ctl.q_empty, (it - 1) & 1, &ctl)) { report_timeout(p, &ctl, 10, (int)item); break; }
                mbar_arrive_expect_tx(smem_u32(&ctl.q_full), NQ * C::TILE_BYTES);
                // in the sorted layout the copies are indexed [head of the batch][sorted slot]
                const int qh = p.sorted ? hq : h, qb = p.sorted ? 0 : b;
                const int kh = p.sorted ? b * p.Hkv + hk : hk;
                for (int x = 0; x < NQ; ++x)
                    for (int c = 0; c < C::SUBT; ++c)
                        tma_load_4d(sq + x * C::TILE_BYTES + c * C::SUB_BYTES, &tm_q, smem_u32(&ctl.q_full), c * 64,
                                    (A * NQ + x) * 128, qh, qb);
                // one K or V tile into the next stage(s) of the ring
                auto load_tile = [&](bool is_v, int tile) {
                    for (int part = 0; part < C::PARTS; ++part) {
                        if (nload == p.stall_at) { ++nload; continue; }      // diagnostic: this stage is never filled
                        const int slot = (int)(nload % C::NSTAGE);
                        const long long use = nload / C::NSTAGE;
                        if (use > 0 && !ctl_wait(&ctl.kv_empty[slot], (uint32_t)((use - 1) & 1), &ctl)) {
                            report_timeout(p, &ctl, 11, (int)item);
                            ok = false;
                            return;
                        }
                        const uint32_t bar = smem_u32(&ctl.kv_full[slot]);
                        const uint32_t dst = skv + slot * C::STAGE_BYTES;
                        mbar_arrive_expect_tx(bar, C::STAGE_BYTES);
                        if (is_v) {     // 128 / PARTS keys x all dimensions: one box of 64 columns x 128 / PARTS rows per sub-tile
                            for (int c = 0; c < C::SUBT; ++c)
                                tma_load_4d(dst + c * (C::SUB_BYTES / C::PARTS), &tm_v, bar, c * 64, tile * 128 + part * (128 / C::PARTS),
                                            kh, qb);
                        } else {        // all keys x D / PARTS dimensions
                            for (int c = 0; c < C::SUBT / C::PARTS; ++c)
                                tma_load_4d(dst + c * C::SUB_BYTES, &tm_k, bar, (part * (C::SUBT / C::PARTS) + c) * 64, tile * 128, kh, qb);
                        }
                        ++nload;
                    }
                };
                if constexpr (C::K_AHEAD) {
                    // load order K(0), then per tile K(next), V(current): the K of the next tile is needed first (its
                    // S is issued before the current P V) and so travels ahead of the V it shares the ring with
                    load_tile(false, kb);
                    while (ok && kb >= 0) {
                        const int nxt = walk.next();
                        if (nxt >= 0) load_tile(false, nxt);
                        if (ok) load_tile(true, kb);
                        kb = nxt;
                    }
                } else {
                    // two query tiles: V(current) is consumed and released before K(next), so it goes first
                    for (; ok && kb >= 0; kb = walk.next()) {
                        load_tile(false, kb);
                        if (ok) load_tile(true, kb);
                    }
                }
                ++it;
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // The whole warp runs the loop (so that addresses and descriptors stay warp-uniform); one elected
        // lane issues the MMAs and commits.
        {
            constexpr uint32_t IDESC_S = idesc_bf16(128, 128, 0, 0);
            constexpr uint32_t IDESC_O = idesc_bf16(128, D, 0, 1);
            long long nuse = 0;             // K/V stages consumed so far
            uint32_t np[2] = {0, 0};        // P tiles consumed per S/P buffer
            uint32_t gs = 0, gp = 0;        // NQ == 1: S tiles issued / P tiles consumed (buffer = count & 1)
            int it = 0;
            bool ok = true;
            const uint64_t qdesc0 = smem_desc_sw128(sq, 16, 1024);
            const uint64_t kvdesc0 = smem_desc_sw128(skv, 16, 1024);             // K tiles: K-major
            const uint64_t vdesc0 = smem_desc_sw128(skv, C::SUB_BYTES / C::PARTS, 1024);     // V tiles: MN-major, 64-column chunks
            // S[buf] = Q_x K^T
            auto issue_s = [&](int x, int buf, int kslot) {
                if (elect_one()) {
                    const uint32_t d = tmem + (buf ? C::COL_S1 : C::COL_S0);
                    const uint64_t ad = qdesc0 + (uint64_t)((x * C::TILE_BYTES) >> 4);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const uint64_t off = (uint64_t)(((ks / 4) * C::SUB_BYTES + (ks % 4) * 32) >> 4);
                        umma_ss(d, ad + off, kvdesc0 + (uint64_t)((kslot * C::STAGE_BYTES) >> 4) + off, IDESC_S, ks > 0);
                    }
                }
            };
            // O_x (+)= P[buf] V
            auto issue_o = [&](int x, int buf, int vslot, bool first) {
                if (elect_one()) {
                    const uint32_t d = tmem + (x ? C::COL_O1 : C::COL_O0);
                    const uint32_t a = tmem + (buf ? C::COL_S1 : C::COL_S0);
                    const uint64_t bd = vdesc0 + (uint64_t)((vslot * C::STAGE_BYTES) >> 4);
                    // split rows: the P of column half h sits at columns 64 h .. 64 h + 31
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        umma_ts(d, a + (C::NSPLIT == 2 ? (ks / 4) * 64 + (ks % 4) * 8 : ks * 8), bd + (uint64_t)((ks * 2048) >> 4),
                                IDESC_O, (!first) || ks > 0);
                }
            };
            auto commit = [&](uint64_t* bar) {
                if (elect_one()) umma_commit(smem_u32(bar));
            };
            // a ring stage goes back to the producer once the MMAs issued so far have completed
            auto release_tile = [&](int slot) { commit(&ctl.kv_empty[slot]); };
            // wait for the next tile of the ring
            auto wait_kv = [&](int& slot, int where, int item) -> bool {
                slot = (int)(nuse % C::NSTAGE);
                if (!ctl_wait(&ctl.kv_full[slot], (uint32_t)((nuse / C::NSTAGE) & 1), &ctl)) {
                    report_timeout(p, &ctl, where, item);
                    return false;
                }
                ++nuse;
                return true;
            };
            // One query tile: S[buf] = Q K^T and O (+)= P[buf] V stage by stage -- wait for the stage, issue the MMAs that
            // read it, hand it back.  The stages are taken in the ring's order: K(next) before V(current).
            auto s_tile = [&](int buf, int where, int item) -> bool {
                constexpr int KS = D / 16 / C::PARTS;            // k-steps per stage
                const uint32_t d = tmem + (buf ? C::COL_S1 : C::COL_S0);
                for (int part = 0; part < C::PARTS; ++part) {
                    int slot;
                    if (!wait_kv(slot, where, item)) return false;
                    tc_fence_after();
                    if (elect_one()) {
#pragma unroll
                        for (int k2 = 0; k2 < KS; ++k2) {
                            const int ks = part * KS + k2;
                            const uint64_t qoff = (uint64_t)(((ks / 4) * C::SUB_BYTES + (ks % 4) * 32) >> 4);
                            const uint64_t koff = (uint64_t)((slot * C::STAGE_BYTES + (k2 / 4) * C::SUB_BYTES + (k2 % 4) * 32) >> 4);
                            umma_ss(d, qdesc0 + qoff, kvdesc0 + koff, IDESC_S, ks > 0);
                        }
                    }
                    release_tile(slot);
                }
                commit(&ctl.s_full[buf]);
                return true;
            };
            auto o_tile = [&](int buf, bool first, int where, int item) -> bool {
                constexpr int KS = 8 / C::PARTS;
                const uint32_t d = tmem + C::COL_O0;
                const uint32_t a = tmem + (buf ? C::COL_S1 : C::COL_S0);
                for (int part = 0; part < C::PARTS; ++part) {
                    int slot;
                    if (!wait_kv(slot, where, item)) return false;
                    tc_fence_after();
                    if (elect_one()) {
#pragma unroll
                        for (int k2 = 0; k2 < KS; ++k2) {
                            const int ks = part * KS + k2;
                            umma_ts(d, a + (C::NSPLIT == 2 ? (ks / 4) * 64 + (ks % 4) * 8 : ks * 8),
                                    vdesc0 + (uint64_t)((slot * C::STAGE_BYTES + k2 * 2048) >> 4), IDESC_O, (!first) || ks > 0);
                        }
                    }
                    release_tile(slot);
                }
                return true;
            };
            Item t;
            for (int round = 0; ok && item_of(p, round, t, (int)gridDim.x, (int)blockIdx.x); ++round) {
                const int A = t.A, hq = t.hq;
                const long long item = t.id;
                TileWalk walk;
                walk.init(p, hq, A * NQ, NQ);
                int cur = walk.next();
                if (cur < 0) continue;
                if (!ctl_wait(&ctl.q_full, it & 1, &ctl)) { report_timeout(p, &ctl, 20, (int)item); break; }
                if constexpr (NQ == 2) {
                    int slot;
                    if (!wait_kv(slot, 21, (int)item)) break;
                    tc_fence_after();
                    issue_s(0, 0, slot); commit(&ctl.s_full[0]);
                    issue_s(1, 1, slot); commit(&ctl.s_full[1]);
                    release_tile(slot);
                } else {
                    if (!s_tile(gs & 1, 21, (int)item)) break;
                    ++gs;
                }
                bool first = true;
                while (cur >= 0) {
                    const int nxt = walk.next();
                    int vslot = 0, kslot = 0;
                    if constexpr (NQ == 2) {
                        // the ring carries V(current) ahead of K(next) here (see the producer)
                        if (!wait_kv(vslot, 22, (int)item)) { ok = false; break; }
                        if (nxt >= 0) {
                            if (!wait_kv(kslot, 23, (int)item)) { ok = false; break; }
                        }
                    }
                    if (nxt < 0) commit(&ctl.q_empty);     // every S of this item has been issued
                    if constexpr (NQ == 2) {
                        // query tile 0
                        if (!ctl_wait(&ctl.p_full[0], np[0] & 1, &ctl)) { report_timeout(p, &ctl, 24, (int)item); ok = false; break; }
                        ++np[0];
                        tc_fence_after();
                        issue_o(0, 0, vslot, first);
                        if (nxt >= 0) { issue_s(0, 0, kslot); commit(&ctl.s_full[0]); }
                        else commit(&ctl.o_full[0]);
                        // query tile 1
                        if (!ctl_wait(&ctl.p_full[1], np[1] & 1, &ctl)) { report_timeout(p, &ctl, 25, (int)item); ok = false; break; }
                        ++np[1];
                        tc_fence_after();
                        issue_o(1, 1, vslot, first);
                        release_tile(vslot);
                        if (nxt >= 0) {
                            issue_s(1, 1, kslot); commit(&ctl.s_full[1]);
                            release_tile(kslot);
                        } else {
                            commit(&ctl.o_full[1]);
                        }
                    } else {
                        // S of the next tile goes to the other buffer before this tile's PV is issued
                        if (nxt >= 0) {
                            if (!s_tile(gs & 1, 23, (int)item)) { ok = false; break; }
                            ++gs;
                        }
                        const int buf = gp & 1;
                        if (!ctl_wait(&ctl.p_full[buf], (gp >> 1) & 1, &ctl)) { report_timeout(p, &ctl, 26, (int)item); ok = false; break; }
                        ++gp;
                        tc_fence_after();
                        if (!o_tile(buf, first, 22, (int)item)) { ok = false; break; }
                        commit(&ctl.pv_done);
                        if (nxt < 0) commit(&ctl.o_full[0]);
                    }
                    first = false;
                    cur = nxt;
                }
                ++it;
            }
        }
        __syncwarp();
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ softmax + epilogue
        reg_inc<REGS_SOFTMAX_2WG>();
        constexpr int NSPLIT = C::NSPLIT, NC = C::NC;
        const int wg = (warp - 4) >> 2;
        const int x = NSPLIT == 2 ? 0 : wg;                  // query tile of this warpgroup
        const int half = NSPLIT == 2 ? wg : 0;               // split rows: its column half of every key tile
        const int row_in_tile = ((warp & 3) << 5) | lane;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_o = tmem + lane_base + (x ? C::COL_O1 : C::COL_O0) + half * (D / 2);   // its part of the O row
        uint32_t nx = 0;                                     // split rows: exchanges done with the partner half
        // logits in log2 units: sl2 * S, or with a softcap sl2 * tanh(cap_in * S)
        const float sl2 = SOFTCAP ? p.softcap * LOG2E : p.scale * LOG2E;
        const float cap_in = SOFTCAP ? p.scale / p.softcap : 0.f;
        uint32_t ns = 0;                                     // S tiles consumed by this warpgroup
        uint32_t ng = 0;                                     // soft gate: tiles whose key assignments this warpgroup has staged
        int it = 0;
        bool ok = true;
        Item t;
        for (int round = 0; ok && item_of(p, round, t, (int)gridDim.x, (int)blockIdx.x); ++round) {
            const int A = t.A, hq = t.hq, bb = t.bb, h = t.h;
            const long long item = t.id;
            const int hk = bb * p.Hkv + h / p.G;
            const int a = A * NQ + x;
            TileWalk walk;
            walk.init(p, hq, A * NQ, NQ);
            int kb = walk.next();
            if (kb < 0) continue;
            // the row's position in the sequence: its index, or in the sorted layout the position its slot holds
            long long i = (long long)a * 128 + row_in_tile;
            int wmin = 0, wmax = 0;
            if (p.sorted) {
                i = __ldg(p.perm_q + (size_t)hq * p.nqp + i);                       // -1 in the padding of a segment
                wmin = __reduce_min_sync(0xffffffffu, i < 0 ? 0x7fffffff : (int)i);
                wmax = __reduce_max_sync(0xffffffffu, (int)i);
            }
            const bool valid = i >= 0 && i < p.n;
            const uint32_t mi = (valid && !p.dense) ? __ldg(p.mq + (size_t)hq * p.n + i) : 0u;
            const uint32_t aq = (!p.dense && !p.sorted && a < p.nqt) ? __ldg(p.andq + (size_t)hq * p.nqt + a) : 0u;
            const long long dfar = (long long)a * 128 - p.w;
            const int f_x = (!p.dense && dfar > 0) ? (int)(dfar / 128) : 0;   // tiles b < f_x are far for this query tile
            float m_used = -INFINITY, l = 0.f;
            bool first = true;
            // soft gate: this row's assignment times lambda / 2 (sigmoid(x) = 1/2 + 1/2 tanh(x / 2))
            constexpr int GQ = GATE ? 2 * GATE : 2;               // 16-byte pieces of an assignment row held per token
            float gi[4 * GQ];
#pragma unroll
            for (int e = 0; e < 4 * GQ; ++e) gi[e] = 0.f;
            if constexpr (GATE != 0) {
                if (valid) {
                    const float4* gp = reinterpret_cast<const float4*>(p.gate_g + ((size_t)bb * p.n + (size_t)i) * p.gate_ld);
#pragma unroll
                    for (int f = 0; f < GQ; ++f) {
                        if (4 * f < p.gate_ld) {
                            const float4 g0 = __ldg(gp + f);
                            gi[4 * f] = g0.x * p.gate_hl; gi[4 * f + 1] = g0.y * p.gate_hl;
                            gi[4 * f + 2] = g0.z * p.gate_hl; gi[4 * f + 3] = g0.w * p.gate_hl;
                        }
                    }
                }
            }
            for (; kb >= 0; kb = walk.next()) {
                TileMask tm;
                if (p.sorted) {
                    const bool share = (mi & __ldg(p.cls_k + (size_t)hk * FOCUS_MAX_CLASSES + walk.jk)) != 0u;
                    build_tile_mask_sorted(tm, p.w, p.perm_k + (size_t)hk * p.nkp + (size_t)kb * 128, share,
                                           valid ? (int)i : -1, wmin, wmax, !p.share_only);
                    if (p.gbits_s && !tm.all_masked)
                        exclude_lower_groups(tm, p.gbits_s + ((size_t)hk * (p.nkp / 128) + kb) * p.K * 4, mi & ((1u << walk.jk) - 1u), p.K);
                } else {
                    build_tile_mask(tm, p, a, kb, i, mi, aq, f_x, hk);
                }
                // ---- soft gate (Eq. 2): the score of a distant pair (i - j > w) is multiplied by sigmoid(lambda g_i . g_j).
                // The warpgroup stages the key assignments of its columns in shared memory before S is needed; every
                // thread then reads them with broadcast 16-byte loads, column by column.
                const unsigned char* gb = nullptr;
                bool gated = false;
                const long long gj0 = (long long)kb * 128 + half * NC;    // first column of this thread's part of the tile
                const long long ifar = i - p.w;                           // columns j < ifar are distant for this row
                if constexpr (GATE != 0) {
                    // the same decision in all four warps of the warpgroup: does the tile hold a distant pair at all
                    const bool tile_gated = !tm.all_masked && ((long long)a * 128 + 127 - p.w > gj0);
                    if (tile_gated) {
                        unsigned char* gw = gate_sm + (wg * 2 + (ng & 1)) * C::GATE_BUF_BYTES;
                        const int col = (warp & 3) * 32 + lane;
                        if (col < NC) {
                            const long long j = gj0 + col;
                            const float4* gp = reinterpret_cast<const float4*>(p.gate_g + ((size_t)bb * p.n + (size_t)(j < p.n ? j : p.n - 1)) * p.gate_ld);
#pragma unroll
                            for (int f = 0; f < GQ; ++f)
                                reinterpret_cast<float4*>(gw + col * C::GATE_ROW_BYTES)[f] = 4 * f < p.gate_ld ? __ldg(gp + f) : make_float4(0.f, 0.f, 0.f, 0.f);
                        }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&ctl.gbar[wg]));
                        if (!ctl_wait(&ctl.gbar[wg], ng & 1, &ctl)) { report_timeout(p, &ctl, 37, (int)item); ok = false; break; }
                        ++ng;
                        gb = gw;
                        gated = __any_sync(0xffffffffu, valid && ifar > gj0);
                    }
                }
                // ---- wait for S
                const int buf = NQ == 2 ? x : (int)(ns & 1);
                const uint32_t par = NQ == 2 ? (ns & 1) : ((ns >> 1) & 1);
                if (!ctl_wait(&ctl.s_full[buf], par, &ctl)) { report_timeout(p, &ctl, 30 + x, (int)item); ok = false; break; }
                // this thread's NC S columns; its packed P columns overwrite the first half of them
                const uint32_t t_s = tmem + lane_base + (buf ? C::COL_S1 : C::COL_S0) + half * NC;
                tc_fence_after();
                uint32_t pk[NC / 2];
                if (tm.all_masked) {
#pragma unroll
                    for (int c = 0; c < NC / 2; ++c) pk[c] = 0u;
                } else {
                    uint32_t sr[NC];
#pragma unroll
                    for (int c = 0; c < NC / 32; ++c) {
                        tmem_ld32(t_s + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[c * 32]));
                        if constexpr (GATE != 0) {       // chunk by chunk: 32 scores, then their factors
                            tmem_wait_ld();
                            if (gated) {
                                const bool wide = p.gate_ld == 8;
                                const int nfar = (int)(ifar - gj0 < 0 ? 0 : (ifar - gj0 > NC ? NC : ifar - gj0));   // columns < nfar are distant
#pragma unroll
                                for (int e0 = 0; e0 < 32; e0 += 4) {        // four columns in flight
                                    float arg[4];
                                    if constexpr (GATE == 1) {
                                        float4 k0[4], k1[4];
#pragma unroll
                                        for (int u = 0; u < 4; ++u) {
                                            const float4* kp = reinterpret_cast<const float4*>(gb + (c * 32 + e0 + u) * 32);
                                            k0[u] = kp[0];
                                            k1[u] = wide ? kp[1] : make_float4(0.f, 0.f, 0.f, 0.f);
                                        }
#pragma unroll
                                        for (int u = 0; u < 4; ++u) {
                                            float2 acc = __fmul2_rn(make_float2(gi[0], gi[1]), make_float2(k0[u].x, k0[u].y));
                                            acc = __ffma2_rn(make_float2(gi[2], gi[3]), make_float2(k0[u].z, k0[u].w), acc);
                                            if (wide) {
                                                float2 acb = __fmul2_rn(make_float2(gi[4], gi[5]), make_float2(k1[u].x, k1[u].y));
                                                acb = __ffma2_rn(make_float2(gi[6], gi[7]), make_float2(k1[u].z, k1[u].w), acb);
                                                acc = __fadd2_rn(acc, acb);
                                            }
                                            arg[u] = acc.x + acc.y;
                                        }
                                    } else {
                                        // longer assignments: piece by piece, two sums per column
                                        float2 acc[4], acb[4];
#pragma unroll
                                        for (int u = 0; u < 4; ++u) acc[u] = acb[u] = make_float2(0.f, 0.f);
#pragma unroll
                                        for (int f = 0; f < GQ; ++f) {
                                            float4 kf[4];
#pragma unroll
                                            for (int u = 0; u < 4; ++u)
                                                kf[u] = reinterpret_cast<const float4*>(gb + (c * 32 + e0 + u) * C::GATE_ROW_BYTES)[f];
#pragma unroll
                                            for (int u = 0; u < 4; ++u) {
                                                acc[u] = __ffma2_rn(make_float2(gi[4 * f], gi[4 * f + 1]), make_float2(kf[u].x, kf[u].y), acc[u]);
                                                acb[u] = __ffma2_rn(make_float2(gi[4 * f + 2], gi[4 * f + 3]), make_float2(kf[u].z, kf[u].w), acb[u]);
                                            }
                                        }
#pragma unroll
                                        for (int u = 0; u < 4; ++u) arg[u] = (acc[u].x + acc[u].y) + (acb[u].x + acb[u].y);
                                    }
#pragma unroll
                                    for (int u = 0; u < 4; ++u) {
                                        const float gate = fmaf(tanh_approx(arg[u]), 0.5f, 0.5f);
                                        const float sv = __uint_as_float(sr[c * 32 + e0 + u]);
                                        sr[c * 32 + e0 + u] = __float_as_uint(c * 32 + e0 + u < nfar ? sv * gate : sv);
                                    }
                                }
                            }
                        }
                    }
                    tmem_wait_ld();
                    if (SOFTCAP) {
#pragma unroll
                        for (int c = 0; c < NC; ++c) sr[c] = __float_as_uint(tanh_approx(__uint_as_float(sr[c]) * cap_in));
                    }
                    if (tm.masked) {
#pragma unroll
                        for (int c = 0; c < NC; ++c)
                            sr[c] = ((tm.kw[(NSPLIT == 2 ? half * 2 : 0) + (c >> 5)] >> (c & 31)) & 1u) ? sr[c] : 0xff800000u;      // -inf
                    }
                    // ---- row maximum of the tile: four independent chains of three-input maxima
                    float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                    for (int c = 0; c < NC; c += 8) {
                        mx0 = max3(mx0, __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]));
                        mx1 = max3(mx1, __uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3]));
                        mx2 = max3(mx2, __uint_as_float(sr[c + 4]), __uint_as_float(sr[c + 5]));
                        mx3 = max3(mx3, __uint_as_float(sr[c + 6]), __uint_as_float(sr[c + 7]));
                    }
                    float mraw = max3(mx0, mx1, fmaxf(mx2, mx3));
                    if constexpr (NSPLIT == 2) {
                        // the two threads of a row exchange the maxima of their halves and then take the same decisions
                        const int par = (int)(nx & 1);
                        const __nv_bfloat16 mine = __float2bfloat16_rn(mraw);
                        xval(par, half, row_in_tile) = mine;
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&ctl.xchg[warp & 3]));
                        if (!ctl_wait(&ctl.xchg[warp & 3], (uint32_t)par, &ctl)) { report_timeout(p, &ctl, 36, (int)item); ok = false; }
                        mraw = fmaxf(__bfloat162float(mine), __bfloat162float(xval(par, half ^ 1, row_in_tile)));
                        ++nx;
                    }
                    const float mt = mraw * sl2;                     // log2 units (sl2 > 0; -inf stays -inf)
                    // ---- lazy maximum: raise the reference only when it lags by more than the threshold
                    float factor = 1.f;
                    bool raise = false;
                    if (m_used == -INFINITY) {
                        m_used = mt;                                 // nothing accumulated yet for this row
                    } else if (mt > m_used + RESCALE_THRESHOLD) {
                        factor = ex2_approx(m_used - mt);
                        m_used = mt;
                        raise = true;
                    }
                    if (__any_sync(0xffffffffu, raise) && !first) {
                        // O may only be touched once the previous PV of this query tile has completed.  With two
                        // query tiles its commit precedes s_full; with double-buffered S it has its own barrier.
                        bool pv_ok = true;
                        if constexpr (NQ == 1) pv_ok = ctl_wait(&ctl.pv_done, (ns - 1) & 1, &ctl);
                        if (!pv_ok) { report_timeout(p, &ctl, 35, (int)item); ok = false; }
                        tc_fence_after();
#pragma unroll 1
                        for (int c = 0; c < D / 16 / NSPLIT; ++c) {      // this thread's part of the O row
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
                    // ---- probabilities: packed fp32 pairs; part of the exponentials on the FMA/ALU pipes
                    const float2 sl2v = make_float2(sl2, sl2), nmv = make_float2(-msub, -msub);
                    float2 acc[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[e] = make_float2(0.f, 0.f);
#pragma unroll
                    for (int c = 0; c < NC; c += 8) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float2 xv = __ffma2_rn(make_float2(__uint_as_float(sr[c + 2 * e]),
                                                                     __uint_as_float(sr[c + 2 * e + 1])), sl2v, nmv);
                            float2 pr;
                            if (e >= 4 - EX2_POLY_PER_8 / 2) {
                                pr = ex2_poly2(xv);
                            } else {
                                pr.x = ex2_approx(xv.x);
                                pr.y = ex2_approx(xv.y);
                            }
                            acc[e] = __fadd2_rn(acc[e], pr);
                            pk[(c >> 1) + e] = pack_bf16x2(pr.x, pr.y);
                        }
                    }
                    l += (acc[0].x + acc[0].y) + (acc[1].x + acc[1].y) + ((acc[2].x + acc[2].y) + (acc[3].x + acc[3].y));
                }
#pragma unroll
                for (int c = 0; c < NC / 64; ++c) tmem_st32(t_s + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&pk[c * 32]));
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(smem_u32(&ctl.p_full[buf]));
                ++ns;
                first = false;
                if (!ok) break;
            }
            if (!ok) break;
            // ---- epilogue: O / l -> bf16 -> global, lse
            if constexpr (NSPLIT == 2) {
                // the two halves add their row sums: two exchanges, the leading bf16 part of the sum and its remainder
                float other = 0.f, rest = l;
                bool xok = true;
                for (int piece = 0; piece < 2 && xok; ++piece) {
                    const int par = (int)(nx & 1);
                    const __nv_bfloat16 mine = __float2bfloat16_rn(rest);
                    rest -= __bfloat162float(mine);
                    xval(par, half, row_in_tile) = mine;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctl.xchg[warp & 3]));
                    xok = ctl_wait(&ctl.xchg[warp & 3], (uint32_t)par, &ctl);
                    other += __bfloat162float(xval(par, half ^ 1, row_in_tile));
                    ++nx;
                }
                if (!xok) { report_timeout(p, &ctl, 38, (int)item); break; }
                l += other;
            }
            if (!ctl_wait(&ctl.o_full[x], it & 1, &ctl)) { report_timeout(p, &ctl, 40 + x, (int)item); break; }
            tc_fence_after();
            const float inv_l = l > 0.f ? 1.f / l : 0.f;        // a row without any pair (possible in a partial pass): zeros, lse = -inf
            __nv_bfloat16* orow = p.o + (size_t)bb * p.o_sb + (size_t)h * p.o_sh + (size_t)(valid ? i : 0) * p.o_sn +
                                  half * (D / 2);
#pragma unroll 1
            for (int c = 0; c < D / 32 / NSPLIT; ++c) {
                uint32_t ov[32];
                tmem_ld32(t_o + c * 32, ov);
                tmem_wait_ld();
                if (valid && p.o32) {
                    float* o32row = p.o32 + ((size_t)hq * p.n + (size_t)i) * D + half * (D / 2) + c * 32;
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
            if (valid && half == 0) p.lse[(size_t)hq * p.n + i] = (m_used + lg2_approx(l)) * LN2;
            tc_fence_before();
            ++it;
        }
    }
    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*(volatile int*)&ctl.abort_flag) {
        // a role gave up: let copies that were already issued land before the CTA leaves
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 20000ull) { }
    }
    if (warp == 1) tmem_dealloc(tmem, 512);
}

template <int D, bool SOFTCAP, int GATE>
static int launch_attn_t(const AttnArgs& a, cudaStream_t st) {
    using C = AttnCfg<D, GATE>;
    CUtensorMap tq, tk, tv;
    int rc;
    const bool sorted = a.ws && !a.local_pass && layout_is_sorted(a.L.layout);
    if (sorted) {
        // gather Q, K, V into the sorted order kept in the workspace; the kernel reads the copies
        char* ws = const_cast<char*>(a.ws);
        if ((rc = launch_gather_sorted(&a.s, a.q, a.s.Hq, true, a.L, a.ws, ws + a.L.qs, st))) return rc;
        if ((rc = launch_gather_sorted(&a.s, a.k, a.s.Hkv, false, a.L, a.ws, ws + a.L.ks, st))) return rc;
        if ((rc = launch_gather_sorted(&a.s, a.v, a.s.Hkv, false, a.L, a.ws, ws + a.L.vs, st))) return rc;
        const int HQ = a.s.batch * a.s.Hq, HK = a.s.batch * a.s.Hkv;
        const focus_tensor sq_t{ws + a.L.qs, (int64_t)HQ * a.L.nqp * D, (int64_t)a.L.nqp * D, D};
        const focus_tensor sk_t{ws + a.L.ks, (int64_t)HK * a.L.nkp * D, (int64_t)a.L.nkp * D, D};
        const focus_tensor sv_t{ws + a.L.vs, (int64_t)HK * a.L.nkp * D, (int64_t)a.L.nkp * D, D};
        if ((rc = make_tmap_qkv(&tq, sq_t, 1, HQ, a.L.nqp, D))) return rc;
        if ((rc = make_tmap_qkv(&tk, sk_t, 1, HK, a.L.nkp, D))) return rc;
        if ((rc = make_tmap_qkv(&tv, sv_t, 1, HK, a.L.nkp, D, 128 / C::PARTS))) return rc;
    } else {
        if ((rc = make_tmap_qkv(&tq, a.q, a.s.batch, a.s.Hq, a.s.n, D))) return rc;
        if ((rc = make_tmap_qkv(&tk, a.k, a.s.batch, a.s.Hkv, a.s.n, D))) return rc;
        if ((rc = make_tmap_qkv(&tv, a.v, a.s.batch, a.s.Hkv, a.s.n, D, 128 / C::PARTS))) return rc;
    }
    AttnParams p;
    p.B = a.s.batch; p.Hq = a.s.Hq; p.Hkv = a.s.Hkv; p.G = a.s.Hq / a.s.Hkv; p.n = a.s.n; p.w = a.s.window; p.K = a.s.K;
    p.nqb = cdiv(a.s.n, 128 * C::NQ);
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
    p.ipb = 2 / C::NQ;
    p.perm_q = sorted ? reinterpret_cast<const int32_t*>(a.ws + a.L.perm_q) : nullptr;
    p.perm_k = sorted ? reinterpret_cast<const int32_t*>(a.ws + a.L.perm_k) : nullptr;
    p.cls_k = sorted ? reinterpret_cast<const uint32_t*>(a.ws + a.L.cls_k) : nullptr;
    p.ncls_k = sorted ? reinterpret_cast<const int32_t*>(a.ws + a.L.ncls_k) : nullptr;
    p.qrange = sorted ? reinterpret_cast<const int32_t*>(a.ws + a.L.qrange) : nullptr;
    p.order = sorted ? reinterpret_cast<const int32_t*>(a.ws + a.L.order) : nullptr;
    p.counters = a.ws ? reinterpret_cast<const unsigned long long*>(a.ws + a.L.counters) : nullptr;
    p.gate_g = a.gate_g; p.gate_ld = a.gate_ld; p.gate_hl = 0.5f * a.gate_lambda;
    p.local_only = a.local_pass ? 1 : 0;
    p.share_only = (sorted && layout_has_window_pass(a.L.layout)) ? 1 : 0;
    p.gbits_s = (sorted && a.L.layout == FOCUS_LAYOUT_GROUP_MAJOR) ? reinterpret_cast<const uint32_t*>(a.ws + a.L.gbits_s) : nullptr;
    p.o32 = a.o32;
    p.wait_limit_ns = a.wait_limit_ns;
    p.stall_at = a.stall_at;
    if (sorted) p.nitems = (long long)a.s.batch * a.s.Hq * p.nqblk * p.ipb;
    int dev = 0, sms = 0;
    if ((rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice"))) return rc;
    if ((rc = check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "cudaDeviceGetAttribute"))) return rc;
    auto kern = focus_attn_kernel<D, SOFTCAP, GATE>;
    if ((rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM_BYTES),
                         "cudaFuncSetAttribute(attn)")))
        return rc;
    const int grid = (int)(p.nitems < sms ? p.nitems : sms);
    kern<<<grid, C::THREADS, C::SMEM_BYTES, st>>>(tq, tk, tv, p);
    return check_cuda(cudaGetLastError(), "attention kernel launch");
}

static int launch_attn_one(const AttnArgs& a, cudaStream_t st);

int launch_attn_sm100(const AttnArgs& a, cudaStream_t st) {
    if (a.ws && layout_has_window_pass(a.L.layout) && !a.local_pass) {
        // (1) sharing pairs in the class-sorted order -> o, lse; rows of blocks without key tiles keep lse = -inf
        // (2) window-only pairs in token order -> workspace; (3) join through the logsumexps
        char* ws = const_cast<char*>(a.ws);
        const size_t rows = (size_t)a.s.batch * a.s.Hq * a.s.n;
        int rc = launch_fill_f32(a.lse, rows, -INFINITY, st);
        if (rc) return rc;
        AttnArgs s1 = a;
        s1.o32 = reinterpret_cast<float*>(ws + a.L.o_sorted);
        if ((rc = launch_attn_one(s1, st))) return rc;
        AttnArgs s2 = a;
        s2.local_pass = true;
        s2.o32 = reinterpret_cast<float*>(ws + a.L.o_local);
        s2.lse = reinterpret_cast<float*>(ws + a.L.lse_local);
        if ((rc = launch_attn_one(s2, st))) return rc;
        return launch_merge_partials(&a.s, a.o, a.lse, s1.o32, s2.o32, s2.lse, st);
    }
    return launch_attn_one(a, st);
}

static int launch_attn_one(const AttnArgs& a, cudaStream_t st) {
    const bool cap = a.s.softcap > 0.f;
    if (a.gate_g) {      // training-time gated forward: dense causal walk, no softcap
        const int chunks = a.gate_ld <= 8 ? 1 : a.gate_ld / 8;      // 8-float chunks of an assignment row
        switch (a.s.D) {
            case 64: return chunks == 1 ? launch_attn_t<64, false, 1>(a, st) : chunks == 2 ? launch_attn_t<64, false, 2>(a, st) : launch_attn_t<64, false, 4>(a, st);
            case 128: return chunks == 1 ? launch_attn_t<128, false, 1>(a, st) : chunks == 2 ? launch_attn_t<128, false, 2>(a, st) : launch_attn_t<128, false, 4>(a, st);
            case 256:
                if (chunks == 4) return fail(FOCUS_ERR_UNSUPPORTED, "the gated forward at D = 256 supports K <= 16");
                return chunks == 1 ? launch_attn_t<256, false, 1>(a, st) : launch_attn_t<256, false, 2>(a, st);
        }
    }
    switch (a.s.D) {
        case 64: return cap ? launch_attn_t<64, true, 0>(a, st) : launch_attn_t<64, false, 0>(a, st);
        case 128: return cap ? launch_attn_t<128, true, 0>(a, st) : launch_attn_t<128, false, 0>(a, st);
        case 256: return cap ? launch_attn_t<256, true, 0>(a, st) : launch_attn_t<256, false, 0>(a, st);
    }
    return fail(FOCUS_ERR_UNSUPPORTED, "D (%d) must be 64, 128 or 256", a.s.D);
}

}  // namespace focus
