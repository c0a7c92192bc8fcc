// focus_decode_step: one new query token per head against the cached keys and values, under the
// same rule as the forward pass (paper Sec. 2 "Efficiency at inference", Appendix D first equation):
// the new token at position n-1 attends key j when n-1-j <= w or its groups meet the key's groups.
// This is the generation use of the method (the paper evaluates generation but gives no procedure).
//
// HBM-bound: only the K and V rows of attended keys are read, each once per KV head for all the query
// heads that share it.  The keys are split over CTAs and, inside a CTA, over warps that never synchronise
// with one another; the partial (max, sum, O) of every warp is merged by a second kernel.  bf16 operands,
// fp32 accumulation, probabilities rounded to bf16 before P V (as in the forward pass).
#include "common.cuh"

namespace focus {

constexpr int DEC_GMAX = 8;          // query heads per KV head served together (rows of the 16-row MMA tile)
constexpr int DEC_GK = 16;           // keys per warp step
constexpr int DEC_NST = 3;           // stages of a warp's private K/V ring
constexpr float DEC_LOG2E = 1.4426950408889634f;
constexpr float DEC_LN2 = 0.6931471805599453f;

template <int D> struct DecCfg {
    static constexpr int WARPS = D == 256 ? 2 : 4;                 // warps per CTA: two CTAs fit an SM at every D
    static constexpr int ROWB = 2 * D + 16;                        // padded row: conflict-free ldmatrix rows
    static constexpr int STAGE = 2 * DEC_GK * ROWB;                // K rows then V rows of one step
    static constexpr size_t SMEM = (size_t)WARPS * DEC_NST * STAGE;
};

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t dec_pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Every warp works on its own: steps of 16 keys, a private ring of K/V rows in shared memory filled with
// asynchronous copies (a row is copied only when some query head of the group attends the key), no
// CTA-wide barrier in the loop.  The G <= 8 query heads that share the KV head are the rows of a 16-row
// warp-level MMA tile (a tile of the 5th-generation tensor cores needs 64 rows and would be 7/8 padding):
// S = Q K^T with K rows as the column operand, P V with V rows through a transposing matrix load.
// Each warp keeps its own running maximum, sum and O and writes its own partial result.
template <int D>
__global__ void __launch_bounds__(DecCfg<D>::WARPS * 32)
decode_partial_kernel(const __nv_bfloat16* __restrict__ q, int64_t q_sb, int64_t q_sh, const __nv_bfloat16* __restrict__ k,
                      int64_t k_sb, int64_t k_sh, int64_t k_sn, const __nv_bfloat16* __restrict__ v, int64_t v_sb,
                      int64_t v_sh, int64_t v_sn, const uint32_t* __restrict__ mq_new, const uint32_t* __restrict__ mk,
                      int Hq, int Hkv, int G, int n, int w, float scale, float softcap, int nsplit, int groups_per_split,
                      float* __restrict__ part) {
    using C = DecCfg<D>;
    constexpr int VEC = D / 8;                                     // 16-byte pieces per row
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ uint32_t kflag_s[C::WARPS][DEC_NST][DEC_GK];        // per staged key: bit g set when query head g attends it
    const int split = blockIdx.x, bh = blockIdx.y;                 // bh = batch * Hkv + KV head
    const int b = bh / Hkv, hk = bh % Hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, qd = lane & 3;                        // this thread's query head (MMA row) and column pair
    const int last = n - 1;                                        // position of the new token
    const float sl2 = (softcap > 0.f ? softcap : scale) * DEC_LOG2E;   // logits in log2 units: sl2 * S or sl2 * tanh(S scale / cap)
    const float cap_in = softcap > 0.f ? scale / softcap : 0.f;
    unsigned char* ring = smem_raw + (size_t)warp * DEC_NST * C::STAGE;
    const uint32_t ring_u32 = (uint32_t)__cvta_generic_to_shared(ring);

    // rows that are never copied still enter the MMAs (with probability 0): keep them finite
    for (int i = lane; i < DEC_NST * C::STAGE / 16; i += 32) reinterpret_cast<uint4*>(ring)[i] = make_uint4(0, 0, 0, 0);
    __syncwarp();

    // Q as the row operand: rows >= G and rows 8..15 are zero
    uint32_t qa[D / 16][2];
    {
        const __nv_bfloat16* qrow = q + (size_t)b * q_sb + (size_t)(hk * G + (g < G ? g : 0)) * q_sh;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            qa[ks][0] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + qd * 2) : 0u;
            qa[ks][1] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8 + qd * 2) : 0u;
        }
    }
    uint32_t mq_all[DEC_GMAX];                                     // every lane needs all heads' masks to flag its key
#pragma unroll
    for (int gg = 0; gg < DEC_GMAX; ++gg) mq_all[gg] = gg < G ? __ldg(mq_new + (size_t)b * Hq + hk * G + gg) : 0u;

    const __nv_bfloat16* kb = k + (size_t)b * k_sb + (size_t)hk * k_sh;
    const __nv_bfloat16* vb = v + (size_t)b * v_sb + (size_t)hk * v_sh;
    const uint32_t* mkh = mk + (size_t)bh * n;

    // this warp's steps: groups g0 + warp, g0 + warp + WARPS, ... of 16 keys
    const int total_groups = (n + DEC_GK - 1) / DEC_GK;
    const int g_begin = split * groups_per_split;
    const int g_end = min(g_begin + groups_per_split, total_groups);
    const int nsteps = g_begin + warp < g_end ? (g_end - g_begin - warp + C::WARPS - 1) / C::WARPS : 0;
    auto first_key = [&](int step) { return (g_begin + warp + step * C::WARPS) * DEC_GK; };

    // mask word of the key lane % 16 of a step (0 when it is local or past the end: not needed then)
    auto load_mask = [&](int step) {
        const int j = first_key(step) + (lane & 15);
        return (step < nsteps && j <= last && last - j > w) ? __ldg(mkh + j) : 0u;
    };
    // flag the 16 keys of a step and start copying the attended rows into ring stage `st` (16-byte asynchronous
    // copies, 16 consecutive lanes per row); one commit group per call, also when nothing is copied
    auto issue = [&](int step, int st, uint32_t mkj) {
        if (step < nsteps) {
            uint32_t bits = 0;
            const int j0 = first_key(step);
            const int j = j0 + (lane & 15);
            if (j <= last) {
                const bool local = last - j <= w;
#pragma unroll
                for (int gg = 0; gg < DEC_GMAX; ++gg)
                    if (gg < G && (local || (mq_all[gg] & mkj))) bits |= 1u << gg;
            }
            if (lane < DEC_GK) kflag_s[warp][st][lane] = bits;
            unsigned char* dst = ring + (size_t)st * C::STAGE;
#pragma unroll
            for (int i = 0; i < DEC_GK * VEC / 32; ++i) {
                const int idx = i * 32 + lane;
                const int r = idx / VEC, c = idx % VEC;
                const uint32_t rb = __shfl_sync(0xffffffffu, bits, r);
                if (rb) {
                    const uint32_t dk = (uint32_t)__cvta_generic_to_shared(dst + r * C::ROWB + c * 16);
                    const uint32_t dv = dk + DEC_GK * C::ROWB;
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dk), "l"(kb + (size_t)(j0 + r) * k_sn + c * 8) : "memory");
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dv), "l"(vb + (size_t)(j0 + r) * v_sn + c * 8) : "memory");
                }
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    float m_run = -INFINITY, l_run = 0.f;          // of head g (the four threads of a quad hold the same values)
    float o[D / 8][4];
#pragma unroll
    for (int nt = 0; nt < D / 8; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;

    // prologue: NST - 1 steps in flight, the mask words of the next one on their way
#pragma unroll
    for (int st = 0; st < DEC_NST - 1; ++st) issue(st, st, load_mask(st));
    uint32_t mk_ahead = load_mask(DEC_NST - 1);
    for (int step = 0; step < nsteps; ++step) {
        const int st = step % DEC_NST;
        issue(step + DEC_NST - 1, (step + DEC_NST - 1) % DEC_NST, mk_ahead);     // the stage freed by the previous step
        mk_ahead = load_mask(step + DEC_NST);
        asm volatile("cp.async.wait_group %0;" ::"n"(DEC_NST - 1) : "memory");
        __syncwarp();
        // ---- flags of this thread's four keys: 2 qd, 2 qd + 1, 8 + 2 qd, 9 + 2 qd
        const uint2 f01 = *reinterpret_cast<const uint2*>(&kflag_s[warp][st][qd * 2]);
        const uint2 f23 = *reinterpret_cast<const uint2*>(&kflag_s[warp][st][8 + qd * 2]);
        const uint32_t any4 = f01.x | f01.y | f23.x | f23.y;
        if (__any_sync(0xffffffffu, any4 != 0u)) {
            const uint32_t kst = ring_u32 + st * C::STAGE, vst = kst + DEC_GK * C::ROWB;
            // ---- S = Q K^T for 16 keys: two 8-key column tiles
            float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
            {
                const int mi = lane >> 3, mr = lane & 7;           // matrix index and row for the matrix loads
                const uint32_t kaddr = kst + (mr + 8 * (mi >> 1)) * C::ROWB + 16 * (mi & 1);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    uint32_t kr[4];
                    ldmatrix_x4(kr, kaddr + ks * 32);
                    mma_bf16_16816(s0, qa[ks][0], 0u, qa[ks][1], 0u, kr[0], kr[1]);
                    mma_bf16_16816(s1, qa[ks][0], 0u, qa[ks][1], 0u, kr[2], kr[3]);
                }
            }
            // ---- scores of head g for the thread's four keys, in log2 units
            float sc[4] = {s0[0], s0[1], s1[0], s1[1]};
            const uint32_t fl[4] = {f01.x, f01.y, f23.x, f23.y};
            float cm = -INFINITY;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float x = sc[e];
                if (softcap > 0.f) x = tanhf(x * cap_in);
                x = ((fl[e] >> g) & 1u) ? x * sl2 : -INFINITY;
                sc[e] = x;
                cm = fmaxf(cm, x);
            }
            cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 1));
            cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 2));
            const float m_new = fmaxf(m_run, cm);
            const float factor = (m_run == -INFINITY) ? 0.f : exp2f(m_run - m_new);     // nothing accumulated yet: O and l are 0
            float p[4], psum = 0.f;
#pragma unroll
            for (int e = 0; e < 4; ++e) { p[e] = (m_new == -INFINITY) ? 0.f : exp2f(sc[e] - m_new); psum += p[e]; }
            psum += __shfl_xor_sync(0xffffffffu, psum, 1);
            psum += __shfl_xor_sync(0xffffffffu, psum, 2);
            l_run = l_run * factor + psum;
            m_run = m_new;
            const uint32_t pa0 = dec_pack_bf16(p[0], p[1]), pa2 = dec_pack_bf16(p[2], p[3]);
            // ---- O = O * factor + P V
            {
                const int mi = lane >> 3, mr = lane & 7;
                const uint32_t vaddr = vst + (mr + 8 * (mi & 1)) * C::ROWB + 16 * (mi >> 1);
#pragma unroll
                for (int np = 0; np < D / 16; ++np) {
                    uint32_t vr[4];
                    ldmatrix_x4_trans(vr, vaddr + np * 32);
                    o[2 * np][0] *= factor; o[2 * np][1] *= factor;
                    o[2 * np + 1][0] *= factor; o[2 * np + 1][1] *= factor;
                    mma_bf16_16816(o[2 * np], pa0, 0u, pa2, 0u, vr[0], vr[1]);
                    mma_bf16_16816(o[2 * np + 1], pa0, 0u, pa2, 0u, vr[2], vr[3]);
                }
            }
        }
        __syncwarp();                               // the stage may be refilled by the next issue
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    // ---- merge the warps of the CTA (through the ring, no longer needed), then one partial result per split:
    //      [query head][split][2 + D] = (max, sum, O)
    __syncthreads();
    float* xw = reinterpret_cast<float*>(smem_raw);             // [WARPS][GMAX][D + 2]
    if (g < DEC_GMAX) {
        float* dstw = xw + ((size_t)warp * DEC_GMAX + g) * (D + 2);
        if (qd == 0) { dstw[0] = m_run; dstw[1] = l_run; }
#pragma unroll
        for (int nt = 0; nt < D / 8; ++nt)
            *reinterpret_cast<float2*>(dstw + 2 + nt * 8 + qd * 2) = make_float2(o[nt][0], o[nt][1]);
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < G * D; idx += C::WARPS * 32) {
        const int gg = idx / D, d = idx % D;
        float M = -INFINITY;
#pragma unroll
        for (int ww = 0; ww < C::WARPS; ++ww) M = fmaxf(M, xw[((size_t)ww * DEC_GMAX + gg) * (D + 2)]);
        float L = 0.f, acc = 0.f;
#pragma unroll
        for (int ww = 0; ww < C::WARPS; ++ww) {
            const float* src = xw + ((size_t)ww * DEC_GMAX + gg) * (D + 2);
            const float wgt = src[0] == -INFINITY ? 0.f : exp2f(src[0] - M);
            L = fmaf(src[1], wgt, L);
            acc = fmaf(src[2 + d], wgt, acc);
        }
        float* dst = part + (((size_t)b * Hq + hk * G + gg) * nsplit + split) * (D + 2);
        if (d == 0) { dst[0] = M; dst[1] = L; }
        dst[2 + d] = acc;
    }
}

// one block per query head: merge the splits (weights of the splits once through shared memory, then every
// thread one output dimension with independent loads)
__global__ void __launch_bounds__(256)
decode_merge_kernel(const float* __restrict__ part, int nsplit, int D, int Hq, __nv_bfloat16* __restrict__ o, int64_t o_sb,
                    int64_t o_sh, float* __restrict__ lse) {
    __shared__ float wgt_s[512];
    __shared__ float red_s[8];
    const int hq = blockIdx.x, t = threadIdx.x;
    const float* p = part + (size_t)hq * nsplit * (D + 2);
    float m = -INFINITY;
    for (int s = t; s < nsplit; s += 256) m = fmaxf(m, p[(size_t)s * (D + 2)]);
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    if ((t & 31) == 0) red_s[t >> 5] = m;
    __syncthreads();
    float M = red_s[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) M = fmaxf(M, red_s[i]);
    __syncthreads();
    float l = 0.f;
    for (int s = t; s < nsplit; s += 256) {
        const float ms = p[(size_t)s * (D + 2)];
        const float wg = ms == -INFINITY ? 0.f : exp2f(ms - M);
        wgt_s[s] = wg;
        l = fmaf(p[(size_t)s * (D + 2) + 1], wg, l);
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
    if ((t & 31) == 0) red_s[t >> 5] = l;
    __syncthreads();
    float L = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) L += red_s[i];
    for (int d = t; d < D; d += 256) {
        float acc = 0.f;
#pragma unroll 8
        for (int s = 0; s < nsplit; ++s) acc = fmaf(p[(size_t)s * (D + 2) + 2 + d], wgt_s[s], acc);
        o[(size_t)(hq / Hq) * o_sb + (size_t)(hq % Hq) * o_sh + d] = __float2bfloat16(acc / L);
    }
    if (t == 0) lse[hq] = (M + log2f(L)) * DEC_LN2;
}

static int decode_warps(int D) { return D == 256 ? 2 : 4; }

static int decode_splits(const focus_shape* s) {
    const int groups = cdiv(s->n, DEC_GK);
    const int heads = s->batch * s->Hkv;
    int want = cdiv(2 * 148, heads);                 // about two CTAs per SM in total
    const int max_useful = cdiv(groups, 4 * decode_warps(s->D));     // at least four steps per warp
    if (want > max_useful) want = max_useful;
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
    using C = DecCfg<D>;
    const int nsplit = decode_splits(s);
    const int groups = cdiv(s->n, DEC_GK);
    const int gps = cdiv(groups, nsplit);
    auto kern = decode_partial_kernel<D>;
    int rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM),
                        "cudaFuncSetAttribute(decode)");
    if (rc) return rc;
    kern<<<dim3(nsplit, s->batch * s->Hkv), C::WARPS * 32, C::SMEM, st>>>(
        reinterpret_cast<const __nv_bfloat16*>(q.ptr), q.stride_b, q.stride_h, reinterpret_cast<const __nv_bfloat16*>(k.ptr),
        k.stride_b, k.stride_h, k.stride_n, reinterpret_cast<const __nv_bfloat16*>(v.ptr), v.stride_b, v.stride_h, v.stride_n,
        mq_new, mk, s->Hq, s->Hkv, s->Hq / s->Hkv, s->n, s->window, scale, s->softcap, nsplit, gps, part);
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
