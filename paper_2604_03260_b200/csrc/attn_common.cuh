// Pieces shared by the attention kernels (one CTA per SM, and one CTA pair per two SMs): launch parameters, the walk over
// the key tiles an item visits, the per-tile keep bitmaps of the Focus mask (paper Appendix D, first equation), the order
// in which items are handed out.
#pragma once

#include <cuda_fp16.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace focus {

using namespace ptx;

constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;
constexpr float RESCALE_THRESHOLD = 8.0f;   // log2 units: the stale maximum may lag by a factor of 256
// Of every 8 consecutive probabilities, this many take their exponential from a polynomial on the
// FMA/ALU pipes instead of the special-function unit, which would otherwise be as busy as the tensor pipe.
constexpr int EX2_POLY_PER_8 = 0;
// Registers per thread after the warps have split into roles (setmaxnreg): the load/MMA warpgroup
// gives most of its share to the softmax warpgroups.
constexpr int REGS_CONTROL = 96;
constexpr int REGS_SOFTMAX_2WG = 200;        // 128*96 + 256*200 = 63488 <= 65536
constexpr int REGS_SOFTMAX_1WG = 232;        // 128*96 + 128*232 (unused while a single query tile is split over two warpgroups)

__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

// 2^x for a pair of arguments in [-inf, 8] without the special-function unit: split x = n + f with
// n = round(x) (magic-number addition), evaluate a cubic for 2^f on [-0.5, 0.5] (relative error
// 7.5e-5, far below the bf16 rounding of the probabilities) and add n to the exponent field.
// Arguments below -126 (masked pairs arrive as -inf) give 2^-126, which vanishes in every sum.
__device__ __forceinline__ float2 ex2_poly2(float2 x) {
    constexpr float MAGIC = 12582912.f;      // 1.5 * 2^23
    x.x = fmaxf(x.x, -126.f);
    x.y = fmaxf(x.y, -126.f);
    const float2 t = __fadd2_rn(x, make_float2(MAGIC, MAGIC));
    const float2 n = __fadd2_rn(t, make_float2(-MAGIC, -MAGIC));
    const float2 f = __ffma2_rn(n, make_float2(-1.f, -1.f), x);
    float2 p = __ffma2_rn(make_float2(0.0551716648f, 0.0551716648f), f, make_float2(0.2426111251f, 0.2426111251f));
    p = __ffma2_rn(p, f, make_float2(0.6932609677f, 0.6932609677f));
    p = __ffma2_rn(p, f, make_float2(0.9999280572f, 0.9999280572f));
    float2 r;
    r.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23));
    r.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23));
    return r;
}

struct AttnParams {
    int B, Hq, Hkv, G, n, w, K;
    int nqb;                 // items per head: 256-row query blocks (128-row tiles when D = 256)
    int nqt, nkt, nkw;
    int dense;
    float scale, softcap;
    const uint32_t* mq;
    const uint32_t* gbits;
    const uint32_t* live;
    const uint32_t* andq;
    const uint32_t* andk;
    __nv_bfloat16* o;
    int64_t o_sb, o_sh, o_sn;
    float* lse;
    int32_t* status;
    long long nitems;
    // class-sorted layout: Q/K/V are the sorted copies, tiles are tiles of the sorted order
    int sorted;
    int nqp, nkp, nqblk;
    int ipb;                 // items per block of 256 sorted queries (1, or 2 when an item is one query tile)
    const int32_t* perm_q;
    const int32_t* perm_k;
    const uint32_t* cls_k;
    const int32_t* ncls_k;
    const int32_t* qrange;
    const int32_t* order;
    const unsigned long long* counters;
    // training-time soft gate (Sec. 2 "Gated attention"): assignments [B, n, gate_ld] fp32, lambda / 2
    const float* gate_g;
    int gate_ld;
    float gate_hl;
    // window pass of the split layout: only the tiles that reach into the window, only pairs WITHOUT a shared group
    // class-sorted pass of the split layout: only pairs WITH a shared group (the window pass covers the others)
    int share_only;
    // group-major keys: bitmaps of the list entries per group, [B*Hkv][nkp/128][K][4] (nullptr in the other layouts)
    const uint32_t* gbits_s;
    int local_only;
    float* o32;              // partial passes: O in fp32, rows [B*Hq][n][D], instead of bf16 to `o`
    unsigned long long wait_limit_ns;   // bound of every wait inside the kernel
    long long stall_at;      // diagnostic: index of a K/V ring stage the producer leaves unfilled (-1 = none)
};

// Enumerates the key tiles a 256-row query block visits, in increasing order.  Every role of the
// CTA runs the same walk over the same data, which keeps them in step without communication.
struct TileWalk {
    const uint32_t* l0;
    int nl, nkw;                // live rows (query tiles) to OR, and their stride in words
    int f0, b_last, b, wd;
    uint32_t bits;
    bool far_phase;
    // class-sorted layout: the ranges of sorted key tiles, key class by key class
    const int32_t* qr;
    int nck, jk, rend;
    bool sorted;

    // a0 = first 128-row query tile of the item, nq = number of query tiles of the item (1 or 2)
    __device__ __forceinline__ void init(const AttnParams& p, int hq, int a0, int nq) {
        sorted = p.sorted != 0;
        if (sorted) {
            const int hk = (hq / p.Hq) * p.Hkv + (hq % p.Hq) / p.G;
            qr = p.qrange + ((size_t)hq * p.nqblk + (a0 >> 1)) * FOCUS_MAX_CLASSES * 2;
            nck = __ldg(p.ncls_k + hk);
            jk = -1;
            b = rend = 0;
            return;
        }
        const long long last_row = min((long long)p.n, (long long)(a0 + nq) * 128) - 1;
        b_last = (int)(last_row / 128);
        f0 = 0;
        l0 = nullptr;
        nl = 0;
        nkw = p.nkw;
        if (!p.dense) {
            const long long d = (long long)a0 * 128 - p.w;
            f0 = d > 0 ? (int)(d / 128) : 0;              // tiles before f0 are far for every query tile of the item
            l0 = p.live + ((size_t)hq * p.nqt + a0) * p.nkw;
            nl = min(nq, p.nqt - a0);
        }
        far_phase = f0 > 0 && !p.local_only;
        wd = -1;
        bits = 0;
        b = f0;
    }
    // next key tile, or -1; in the sorted layout `jk` is then the class index of that tile
    __device__ __forceinline__ int next() {
        if (sorted) {
            while (b >= rend) {
                if (++jk >= nck) return -1;
                b = __ldg(qr + 2 * jk);
                rend = __ldg(qr + 2 * jk + 1);
            }
            return b++;
        }
        if (far_phase) {
            for (;;) {
                if (bits) {
                    const int c = __ffs(bits) - 1;
                    bits &= bits - 1;
                    return wd * 32 + c;
                }
                ++wd;
                if (wd * 32 >= f0) { far_phase = false; break; }
                uint32_t x = 0;
                for (int r = 0; r < nl; ++r) x |= __ldg(l0 + (size_t)r * nkw + wd);
                const int rem = f0 - wd * 32;
                if (rem < 32) x &= (1u << rem) - 1u;
                bits = x;
            }
        }
        if (b <= b_last) return b++;
        return -1;
    }
};

// Per-row 128-bit keep bitmap of one (query tile, key tile) pair.  Returns false when the tile needs
// no mask at all; `all_masked` is set when no pair of the tile can be attended.
struct TileMask {
    uint32_t kw[4];
    bool masked, all_masked;
};

__device__ __forceinline__ void build_tile_mask(TileMask& tm, const AttnParams& p, int a, int kb, long long i,
                                                uint32_t mi, uint32_t aq, int f_x, int hk) {
    const long long c0 = (long long)kb * 128;
    const long long r_first = (long long)a * 128, r_last = r_first + 127;
    tm.all_masked = c0 > r_last || r_first >= p.n;
    const bool need_causal = c0 + 127 > r_first;
    bool need_group = false, need_window = false;
    if (!p.dense && !tm.all_masked) {
        if (p.local_only) {
            need_group = need_window = true;
        } else if (kb < f_x) {
            need_group = !(aq & __ldg(p.andk + (size_t)hk * p.nkt + kb));
        } else if (r_last - c0 > p.w) {
            need_group = need_window = true;
        }
    }
    tm.masked = need_causal || need_group;
    tm.kw[0] = tm.kw[1] = tm.kw[2] = tm.kw[3] = 0xffffffffu;
    if (tm.masked && !tm.all_masked) {
        uint32_t sh[4] = {0, 0, 0, 0};
        if (need_group) {
            const uint32_t* gb = p.gbits + ((size_t)hk * p.nkt + kb) * p.K * 4;
            for (uint32_t rem = mi; rem; rem &= rem - 1) {
                const int g = __ffs(rem) - 1;
                if (g < p.K) {
                    const uint4 t = __ldg(reinterpret_cast<const uint4*>(gb + g * 4));
                    sh[0] |= t.x; sh[1] |= t.y; sh[2] |= t.z; sh[3] |= t.w;
                }
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint32_t keep = 0xffffffffu;
            if (need_group) {
                keep = sh[q];
                if (need_window) {
                    const long long lo = i - p.w - c0 - 32 * q;          // columns >= lo are inside the window
                    const uint32_t win = lo <= 0 ? 0xffffffffu : (lo >= 32 ? 0u : ~((1u << (int)lo) - 1u));
                    keep = p.local_only ? (win & ~keep) : (keep | win);     // window pass: in the window and not sharing
                }
            }
            if (need_causal) {
                const long long nk = i - c0 + 1 - 32 * q;                // columns < nk are causal
                keep &= nk >= 32 ? 0xffffffffu : (nk <= 0 ? 0u : ((1u << (int)nk) - 1u));
            }
            tm.kw[q] = keep;
        }
    }
}

// Item order.  Items are laid out KV head by KV head, heaviest query block first inside a head
// group, so that the CTAs running at the same time stream the K/V of one KV head through L2.  CTA c
// takes position c of every even round of g items and position g-1-c of every odd round, which
// cancels the cost gradient inside a round (g workers: CTAs, or CTA pairs).  Returns false past the last item.
struct Item { int A, bb, h, hq; long long id; };
__device__ __forceinline__ bool item_of(const AttnParams& p, int round, Item& t, int g, int c) {
    t.id = (long long)round * g + ((round & 1) ? g - 1 - c : c);
    if (t.id >= p.nitems) return false;
    if (p.sorted) {
        const long long e = t.id / p.ipb;
        t.hq = __ldg(p.order + 2 * e);
        t.A = __ldg(p.order + 2 * e + 1) * p.ipb + (int)(t.id % p.ipb);
        t.bb = t.hq / p.Hq;
        t.h = t.hq % p.Hq;
        return true;
    }
    const int per_group = p.nqb * p.G;
    const int grp = (int)(t.id / per_group);              // batch * Hkv + KV head
    const int rem = (int)(t.id % per_group);
    t.A = p.nqb - 1 - rem / p.G;
    t.bb = grp / p.Hkv;
    t.h = (grp % p.Hkv) * p.G + rem % p.G;
    t.hq = t.bb * p.Hq + t.h;
    return true;
}

// number of entries of the ascending 128-entry array `a` that are <= v (fixed-depth search)
__device__ __forceinline__ int count_le_128(const int32_t* __restrict__ a, int v) {
    int lo = 0;
#pragma unroll
    for (int step = 64; step >= 1; step >>= 1)
        if (__ldg(a + lo + step - 1) <= v) lo += step;
    return lo + (lo == 127 && __ldg(a + 127) <= v ? 1 : 0);
}

// Tile mask in the class-sorted layout.  The keys of a tile belong to one class and their original
// positions `kpos` ascend, so a row keeps a contiguous range of columns: those at or before its own
// position and, unless the classes share a group, not further back than the window.  The decisions
// "no mask needed" / "nothing attended" are taken per warp from the warp's smallest and largest row
// position.
// `window_ok` = false (class-sorted pass of the split layout): a row that shares no group with the tile's class keeps
// nothing of it, whatever the distance.
__device__ __forceinline__ void build_tile_mask_sorted(TileMask& tm, int w, const int32_t* __restrict__ kpos, bool share,
                                                       int pos, int wmin, int wmax, bool window_ok) {
    const int k_first = __ldg(kpos), k_last = __ldg(kpos + 127);
    tm.all_masked = wmax < 0 || k_first > wmax;
    const bool none = !share && !window_ok;
    // (window_ok is the same for the whole grid, so the vote is skipped or taken by every lane alike)
    const bool any_none = !window_ok && __any_sync(0xffffffffu, none);
    const bool need_causal = k_last > wmin;
    const bool need_window = !share && ((long long)wmax - k_first > w);
    tm.masked = need_causal || need_window || any_none;
    tm.kw[0] = tm.kw[1] = tm.kw[2] = tm.kw[3] = 0xffffffffu;
    if (tm.masked && !tm.all_masked) {
        const int hi = none ? 0 : (need_causal ? (pos < 0 ? 0 : count_le_128(kpos, pos)) : 128);          // columns < hi are causal
        const long long edge = (long long)pos - w - 1;
        const int lo = (need_window && pos >= 0 && edge >= 0) ? count_le_128(kpos, (int)edge) : 0;   // columns >= lo are in the window
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int h = hi - 32 * q, l = lo - 32 * q;
            const uint32_t below_hi = h >= 32 ? 0xffffffffu : (h <= 0 ? 0u : ((1u << h) - 1u));
            const uint32_t below_lo = l >= 32 ? 0xffffffffu : (l <= 0 ? 0u : ((1u << l) - 1u));
            tm.kw[q] = below_hi & ~below_lo;
        }
    }
}

// Group-major keys: the tile belongs to the list of group g.  A key that shares a LOWER group with the row is attended
// under that lower group's list, so here it is masked out: `lower` = the row's groups below g, `gb` = the tile's
// per-group bitmaps.  Every sharing pair is then computed exactly once.
__device__ __forceinline__ void exclude_lower_groups(TileMask& tm, const uint32_t* __restrict__ gb, uint32_t lower, int K) {
    uint32_t ex[4] = {0u, 0u, 0u, 0u};
    for (uint32_t rem = lower; rem; rem &= rem - 1) {
        const int a = __ffs(rem) - 1;
        if (a < K) {
            const uint4 t = __ldg(reinterpret_cast<const uint4*>(gb + a * 4));
            ex[0] |= t.x; ex[1] |= t.y; ex[2] |= t.z; ex[3] |= t.w;
        }
    }
    if (ex[0] | ex[1] | ex[2] | ex[3]) {
        tm.masked = true;
        tm.kw[0] &= ~ex[0]; tm.kw[1] &= ~ex[1]; tm.kw[2] &= ~ex[2]; tm.kw[3] &= ~ex[3];
    }
}


}  // namespace focus
