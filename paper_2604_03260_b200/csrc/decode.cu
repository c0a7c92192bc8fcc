// focus_decode_step: one new query token per head against the cached keys and values, under the
// same rule as the forward pass (paper Sec. 2 "Efficiency at inference", Appendix C first equation):
// the new token at position n-1 attends key j when n-1-j <= w or its groups meet the key's groups.
// This is the generation use of the method (the paper evaluates generation but gives no procedure).
//
// HBM-bound: only the K and V rows of attended keys are read.  Split over the keys: a CTA owns a
// range of keys of one KV head and serves the G query heads that share it; per chunk of 128 keys the
// attended rows are copied to shared memory (coalesced asynchronous 16-byte copies, skipped row by
// row when no query head of the group attends the key), thread = key computes the G scores, thread =
// output dimension accumulates P V; the partial (max, sum, O) of every split is merged by a second
// kernel.  fp32 throughout on the exact bf16 values; probabilities are not rounded.
#include "common.cuh"

namespace focus {

constexpr int DEC_KEYS = 128;        // keys per chunk
constexpr int DEC_THREADS = 2 * DEC_KEYS;   // two threads per key for the scores (half of the query heads each);
                                            // for P V: DEC_ROWGROUPS groups of keys x 64 dimension slots
constexpr int DEC_NW = DEC_KEYS / 32;       // warps that share one half of the query heads
constexpr int DEC_ROWGROUPS = DEC_THREADS / 64;
constexpr int DEC_ROWS_PER_GROUP = DEC_KEYS / DEC_ROWGROUPS;
constexpr int DEC_GMAX = 8;          // query heads per KV head served by one CTA
constexpr float DEC_LOG2E = 1.4426950408889634f;
constexpr float DEC_LN2 = 0.6931471805599453f;

template <int D>
__global__ void __launch_bounds__(DEC_THREADS)
decode_partial_kernel(const __nv_bfloat16* __restrict__ q, int64_t q_sb, int64_t q_sh, const __nv_bfloat16* __restrict__ k,
                      int64_t k_sb, int64_t k_sh, int64_t k_sn, const __nv_bfloat16* __restrict__ v, int64_t v_sb,
                      int64_t v_sh, int64_t v_sn, const uint32_t* __restrict__ mq_new, const uint32_t* __restrict__ mk,
                      int Hq, int Hkv, int G, int n, int w, float scale, float softcap, int nsplit, int chunks_per_split,
                      float* __restrict__ part) {
    constexpr int ROWB = 2 * D + 16;                 // padded row: conflict-free 16-byte reads per key
    constexpr int VEC = D / 8;                       // 16-byte pieces per row
    constexpr int DPT = D / 64;                      // output dimensions per thread (64 threads span a row)
    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned char* kt = smem_raw;                                  // [128][ROWB]
    unsigned char* vt = kt + DEC_KEYS * ROWB;                   // [128][ROWB]
    float* qs = reinterpret_cast<float*>(vt + DEC_KEYS * ROWB); // [GMAX][D]
    float* ps = qs + DEC_GMAX * D;                                 // [GMAX][128] probabilities of the chunk
    float* red = ps + DEC_GMAX * DEC_KEYS;                      // [GMAX][DEC_NW] per-warp partial maxima / sums
    __shared__ __align__(16) uint32_t keep_s[2][DEC_KEYS];      // per key: bit g set when query head g attends it

    const int split = blockIdx.x, bh = blockIdx.y;                 // bh = batch * Hkv + KV head
    const int b = bh / Hkv, hk = bh % Hkv;
    const int t = threadIdx.x, lane = t & 31;
    const int key = t & (DEC_KEYS - 1);            // the key of the chunk this thread scores
    const int gh = t / DEC_KEYS;                   // ... for the query heads [g_lo, g_hi)
    const int warp = (t >> 5) % DEC_NW;            // warp index among the warps that share gh
    const int GH = (G + 1) / 2;
    const int g_lo = gh * GH, g_hi = min(G, g_lo + GH);
    const int last = n - 1;                                        // position of the new token
    const float sl2 = (softcap > 0.f ? softcap : scale) * DEC_LOG2E;   // logits in log2 units: sl2 * S or sl2 * tanh(S scale / cap)
    const float cap_in = softcap > 0.f ? scale / softcap : 0.f;

    for (int i = t; i < G * D; i += DEC_THREADS) {
        const int g = i / D, d = i % D;
        qs[i] = __bfloat162float(q[(size_t)b * q_sb + (size_t)(hk * G + g) * q_sh + d]);
    }
    // rows that are never copied are still multiplied by probability 0: keep them finite
    for (int i = t; i < DEC_KEYS * ROWB / 16; i += DEC_THREADS) reinterpret_cast<uint4*>(vt)[i] = make_uint4(0, 0, 0, 0);
    uint32_t mqg[DEC_GMAX];
#pragma unroll
    for (int g = 0; g < DEC_GMAX; ++g) mqg[g] = g < G ? __ldg(mq_new + (size_t)b * Hq + hk * G + g) : 0u;

    float m_run[DEC_GMAX], l_run[DEC_GMAX], o_acc[DEC_GMAX][DPT];
#pragma unroll
    for (int g = 0; g < DEC_GMAX; ++g) {
        m_run[g] = -INFINITY; l_run[g] = 0.f;
#pragma unroll
        for (int e = 0; e < DPT; ++e) o_acc[g][e] = 0.f;
    }
    const __nv_bfloat16* kb = k + (size_t)b * k_sb + (size_t)hk * k_sh;
    const __nv_bfloat16* vb = v + (size_t)b * v_sb + (size_t)hk * v_sh;
    const uint32_t* mkh = mk + (size_t)bh * n;

    // mask word of key j (loaded two chunks ahead of its use, so that its latency is never waited for)
    auto load_mask = [&](int j) { return (j <= last && last - j > w) ? __ldg(mkh + j) : 0u; };
    // which query heads attend key j, given its mask word
    auto keep_of = [&](int j, uint32_t mkj) {
        uint32_t keep = 0;
        if (j <= last) {
            const bool local = last - j <= w;
#pragma unroll
            for (int g = 0; g < DEC_GMAX; ++g)
                if (g < G && (local || (mqg[g] & mkj))) keep |= 1u << g;
        }
        return keep;
    };
    // copy the attended rows of a chunk: 16 consecutive threads copy one row; one commit group per call
    auto copy_rows = [&](const __nv_bfloat16* src, int64_t sn, unsigned char* dst, int j0, const uint32_t* flags) {
#pragma unroll
        for (int i = 0; i < VEC / 2; ++i) {
            const int qd = i * DEC_THREADS + t;
            const int r = qd / VEC, c = qd % VEC;
            if (flags[r]) {
                const uint32_t da = (uint32_t)__cvta_generic_to_shared(dst + r * ROWB + c * 16);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(da), "l"(src + (size_t)(j0 + r) * sn + c * 8) : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    const int c_begin = split * chunks_per_split;
    const int c_end = min(c_begin + chunks_per_split, (n + DEC_KEYS - 1) / DEC_KEYS);
    // Pipeline: K of chunk c+1 is copied while P V of chunk c runs, V of chunk c while its scores are computed.
    uint32_t keep = 0;
    uint32_t mk_ahead = 0;                         // mask word of this thread's key in the next chunk
    if (c_begin < c_end) {
        keep = keep_of(c_begin * DEC_KEYS + key, load_mask(c_begin * DEC_KEYS + key));
        keep_s[c_begin & 1][key] = keep;           // both threads of a key write the same word
        if (c_begin + 1 < c_end) mk_ahead = load_mask((c_begin + 1) * DEC_KEYS + key);
    }
    __syncthreads();
    if (c_begin < c_end) copy_rows(kb, k_sn, kt, c_begin * DEC_KEYS, keep_s[c_begin & 1]);
    for (int ch = c_begin; ch < c_end; ++ch) {
        const int j0 = ch * DEC_KEYS;
        const uint32_t* flags = keep_s[ch & 1];
        copy_rows(vb, v_sn, vt, j0, flags);                 // V tile is free: the previous P V ended with a barrier
        uint32_t keep_next = 0;
        if (ch + 1 < c_end) {
            keep_next = keep_of(j0 + DEC_KEYS + key, mk_ahead);
            keep_s[(ch + 1) & 1][key] = keep_next;
            if (ch + 2 < c_end) mk_ahead = load_mask(j0 + 2 * DEC_KEYS + key);
        }
        asm volatile("cp.async.wait_group 1;" ::: "memory");   // K of this chunk has landed
        __syncthreads();
        // ---- thread = (key, half of the query heads): scores, packed pairs (even dims in .x, odd dims in .y)
        float sc[DEC_GMAX];
#pragma unroll
        for (int g = 0; g < DEC_GMAX; ++g) sc[g] = 0.f;
        if (keep) {
            float2 s2[DEC_GMAX / 2 + 1];
#pragma unroll
            for (int gg = 0; gg < DEC_GMAX / 2 + 1; ++gg) s2[gg] = make_float2(0.f, 0.f);
            const unsigned char* row = kt + key * ROWB;
#pragma unroll 4
            for (int vv = 0; vv < VEC; ++vv) {
                const uint4 rv = *reinterpret_cast<const uint4*>(row + vv * 16);
                const uint32_t wds[4] = {rv.x, rv.y, rv.z, rv.w};
                float2 x[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) x[e] = make_float2(__uint_as_float(wds[e] << 16), __uint_as_float(wds[e] & 0xffff0000u));
#pragma unroll
                for (int gg = 0; gg < DEC_GMAX / 2 + 1; ++gg) {
                    const int g = g_lo + gg;
                    if (gg < GH && g < G) {
                        const float4 a0 = *reinterpret_cast<const float4*>(qs + g * D + vv * 8);
                        const float4 a1 = *reinterpret_cast<const float4*>(qs + g * D + vv * 8 + 4);
                        float2 acc = s2[gg];
                        acc = __ffma2_rn(x[0], make_float2(a0.x, a0.y), acc);
                        acc = __ffma2_rn(x[1], make_float2(a0.z, a0.w), acc);
                        acc = __ffma2_rn(x[2], make_float2(a1.x, a1.y), acc);
                        acc = __ffma2_rn(x[3], make_float2(a1.z, a1.w), acc);
                        s2[gg] = acc;
                    }
                }
            }
#pragma unroll
            for (int gg = 0; gg < DEC_GMAX / 2 + 1; ++gg)
#pragma unroll
                for (int g = 0; g < DEC_GMAX; ++g)
                    if (g == g_lo + gg) sc[g] = s2[gg].x + s2[gg].y;
        }
        // ---- per query head: chunk maximum, running maximum, probabilities, running sum
#pragma unroll
        for (int g = 0; g < DEC_GMAX; ++g) {
            if (g >= g_lo && g < g_hi) {
                float s = sc[g];
                if (softcap > 0.f) s = tanhf(s * cap_in);
                s = ((keep >> g) & 1u) ? s * sl2 : -INFINITY;
                sc[g] = s;
                float mx = s;
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
                if (lane == 0) red[g * DEC_NW + warp] = mx;
            }
        }
        __syncthreads();                        // maxima published; K tile no longer read
        if (ch + 1 < c_end) copy_rows(kb, k_sn, kt, j0 + DEC_KEYS, keep_s[(ch + 1) & 1]);
        else asm volatile("cp.async.commit_group;" ::: "memory");      // keep the group count uniform
        float factor[DEC_GMAX], wsum[DEC_GMAX];
#pragma unroll
        for (int g = 0; g < DEC_GMAX; ++g) {
            factor[g] = 1.f; wsum[g] = 0.f;
            if (g < G) {
                float cm = red[g * DEC_NW];
#pragma unroll
                for (int ww = 1; ww < DEC_NW; ++ww) cm = fmaxf(cm, red[g * DEC_NW + ww]);
                const float m_new = fmaxf(m_run[g], cm);
                factor[g] = (m_run[g] == -INFINITY) ? 0.f : exp2f(m_run[g] - m_new);    // nothing accumulated yet: O and l are 0
                m_run[g] = m_new;
                if (g >= g_lo && g < g_hi) {
                    const float pj = (m_new == -INFINITY) ? 0.f : exp2f(sc[g] - m_new);   // -inf score -> 0
                    ps[g * DEC_KEYS + key] = pj;
                    float sum = pj;
#pragma unroll
                    for (int off = 16; off >= 1; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
                    wsum[g] = sum;
                }
            }
        }
        __syncthreads();                        // maxima consumed by everyone
#pragma unroll
        for (int g = 0; g < DEC_GMAX; ++g)
            if (g >= g_lo && g < g_hi && lane == 0) red[g * DEC_NW + warp] = wsum[g];
        asm volatile("cp.async.wait_group 1;" ::: "memory");   // V of this chunk has landed
        __syncthreads();
#pragma unroll
        for (int g = 0; g < DEC_GMAX; ++g)
            if (g < G) {
                float ssum = red[g * DEC_NW];
#pragma unroll
                for (int ww = 1; ww < DEC_NW; ++ww) ssum += red[g * DEC_NW + ww];
                l_run[g] = l_run[g] * factor[g] + ssum;
            }
        // ---- P V: 64 threads span the output dimensions, each group of 64 threads takes its share of the keys
        {
            const int quarter = t >> 6, dp = t & 63;
#pragma unroll
            for (int g = 0; g < DEC_GMAX; ++g)
#pragma unroll
                for (int e = 0; e < DPT; ++e) o_acc[g][e] *= factor[g];
            for (int r = quarter * DEC_ROWS_PER_GROUP; r < (quarter + 1) * DEC_ROWS_PER_GROUP; r += 4) {
                const uint4 kf = *reinterpret_cast<const uint4*>(&flags[r]);
                if (!(kf.x | kf.y | kf.z | kf.w)) continue;              // uniform across the half: none of the four keys attended
                float vv[4][DPT];
#pragma unroll
                for (int rr = 0; rr < 4; ++rr) {
                    const unsigned char* vp = vt + (r + rr) * ROWB + dp * (2 * DPT);
                    if constexpr (DPT == 1) {
                        vv[rr][0] = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(vp));
                    } else if constexpr (DPT == 2) {
                        const uint32_t u = *reinterpret_cast<const uint32_t*>(vp);
                        vv[rr][0] = __uint_as_float(u << 16); vv[rr][1] = __uint_as_float(u & 0xffff0000u);
                    } else {
                        const uint2 u = *reinterpret_cast<const uint2*>(vp);
                        vv[rr][0] = __uint_as_float(u.x << 16); vv[rr][1] = __uint_as_float(u.x & 0xffff0000u);
                        vv[rr][2] = __uint_as_float(u.y << 16); vv[rr][3] = __uint_as_float(u.y & 0xffff0000u);
                    }
                }
#pragma unroll
                for (int g = 0; g < DEC_GMAX; ++g) {
                    if (g < G) {
                        const float4 p4 = *reinterpret_cast<const float4*>(ps + g * DEC_KEYS + r);
#pragma unroll
                        for (int e = 0; e < DPT; ++e) {
                            float a = o_acc[g][e];
                            a = fmaf(p4.x, vv[0][e], a); a = fmaf(p4.y, vv[1][e], a);
                            a = fmaf(p4.z, vv[2][e], a); a = fmaf(p4.w, vv[3][e], a);
                            o_acc[g][e] = a;
                        }
                    }
                }
            }
        }
        __syncthreads();                        // V tile, probabilities and flags of this chunk are free
        keep = keep_next;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    // ---- add the row groups, then the partial result of this split: [query head][split][2 + D] = (max, sum, O)
    __syncthreads();
    float* xch = reinterpret_cast<float*>(kt);              // [row groups - 1][GMAX][D] (the K and V tiles are no longer needed)
    const int quarter = t >> 6, dp = t & 63;
    if (quarter > 0) {
#pragma unroll
        for (int g = 0; g < DEC_GMAX; ++g)
#pragma unroll
            for (int e = 0; e < DPT; ++e) xch[((quarter - 1) * DEC_GMAX + g) * D + dp * DPT + e] = o_acc[g][e];
    }
    __syncthreads();
    if (quarter == 0) {
#pragma unroll
        for (int g = 0; g < DEC_GMAX; ++g) {
            if (g < G) {
                float* dst = part + (((size_t)b * Hq + hk * G + g) * nsplit + split) * (D + 2);
                if (t == 0) { dst[0] = m_run[g]; dst[1] = l_run[g]; }
#pragma unroll
                for (int e = 0; e < DPT; ++e) {
                    float a = o_acc[g][e];
#pragma unroll
                    for (int qq = 0; qq < DEC_ROWGROUPS - 1; ++qq) a += xch[(qq * DEC_GMAX + g) * D + dp * DPT + e];
                    dst[2 + dp * DPT + e] = a;
                }
            }
        }
    }
}

// one block per query head: merge the splits
__global__ void __launch_bounds__(256)
decode_merge_kernel(const float* __restrict__ part, int nsplit, int D, int Hq, __nv_bfloat16* __restrict__ o, int64_t o_sb,
                    int64_t o_sh, float* __restrict__ lse) {
    const int hq = blockIdx.x;
    const float* p = part + (size_t)hq * nsplit * (D + 2);
    float M = -INFINITY;
    for (int s = 0; s < nsplit; ++s) M = fmaxf(M, p[(size_t)s * (D + 2)]);
    float L = 0.f;
    for (int s = 0; s < nsplit; ++s) {
        const float m = p[(size_t)s * (D + 2)];
        if (m != -INFINITY) L += p[(size_t)s * (D + 2) + 1] * exp2f(m - M);
    }
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
        float acc = 0.f;
        for (int s = 0; s < nsplit; ++s) {
            const float m = p[(size_t)s * (D + 2)];
            if (m != -INFINITY) acc = fmaf(p[(size_t)s * (D + 2) + 2 + d], exp2f(m - M), acc);
        }
        o[(size_t)(hq / Hq) * o_sb + (size_t)(hq % Hq) * o_sh + d] = __float2bfloat16(acc / L);
    }
    if (threadIdx.x == 0) lse[hq] = (M + log2f(L)) * DEC_LN2;
}

static int decode_splits(const focus_shape* s) {
    const int chunks = cdiv(s->n, DEC_KEYS);
    const int heads = s->batch * s->Hkv;
    int want = cdiv(4 * 148, heads);                 // about four CTAs per SM in total (two rounds of two resident ones)
    if (want > chunks) want = chunks;
    if (want < 1) want = 1;
    if (want > 512) want = 512;
    return want;
}

size_t decode_workspace_bytes(const focus_shape* s) {
    return (size_t)s->batch * s->Hq * decode_splits(s) * (s->D + 2) * sizeof(float);
}

template <int D>
static int launch_decode_d(const focus_shape* s, const focus_tensor& q, const focus_tensor& k, const focus_tensor& v,
                           const uint32_t* mq_new, const uint32_t* mk, const focus_tensor& o, float* lse, float* part,
                           float scale, cudaStream_t st) {
    const int nsplit = decode_splits(s);
    const int chunks = cdiv(s->n, DEC_KEYS);
    const int cps = cdiv(chunks, nsplit);
    const size_t smem = (size_t)2 * DEC_KEYS * (2 * D + 16) + (size_t)DEC_GMAX * D * 4 + (size_t)DEC_GMAX * DEC_KEYS * 4 +
                        (size_t)DEC_GMAX * DEC_NW * 4;
    auto kern = decode_partial_kernel<D>;
    int rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem),
                        "cudaFuncSetAttribute(decode)");
    if (rc) return rc;
    kern<<<dim3(nsplit, s->batch * s->Hkv), DEC_THREADS, smem, st>>>(
        reinterpret_cast<const __nv_bfloat16*>(q.ptr), q.stride_b, q.stride_h, reinterpret_cast<const __nv_bfloat16*>(k.ptr),
        k.stride_b, k.stride_h, k.stride_n, reinterpret_cast<const __nv_bfloat16*>(v.ptr), v.stride_b, v.stride_h, v.stride_n,
        mq_new, mk, s->Hq, s->Hkv, s->Hq / s->Hkv, s->n, s->window, scale, s->softcap, nsplit, cps, part);
    if ((rc = check_cuda(cudaGetLastError(), "decode kernel launch"))) return rc;
    decode_merge_kernel<<<s->batch * s->Hq, 256, 0, st>>>(part, nsplit, D, s->Hq, reinterpret_cast<__nv_bfloat16*>(o.ptr),
                                                          o.stride_b, o.stride_h, lse);
    return check_cuda(cudaGetLastError(), "decode merge kernel launch");
}

int launch_decode(const focus_shape* s, const focus_tensor& q, const focus_tensor& k, const focus_tensor& v,
                  const uint32_t* mq_new, const uint32_t* mk, const focus_tensor& o, float* lse, float* part, float scale,
                  cudaStream_t st) {
    if (s->Hq / s->Hkv > DEC_GMAX)
        return fail(FOCUS_ERR_UNSUPPORTED, "decode: more than %d query heads per KV head", DEC_GMAX);
    switch (s->D) {
        case 64: return launch_decode_d<64>(s, q, k, v, mq_new, mk, o, lse, part, scale, st);
        case 128: return launch_decode_d<128>(s, q, k, v, mq_new, mk, o, lse, part, scale, st);
        case 256: return launch_decode_d<256>(s, q, k, v, mq_new, mk, o, lse, part, scale, st);
    }
    return fail(FOCUS_ERR_UNSUPPORTED, "D (%d) must be 64, 128 or 256", s->D);
}

}  // namespace focus
