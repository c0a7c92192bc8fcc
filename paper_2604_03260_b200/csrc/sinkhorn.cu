// focus_sinkhorn: the Sinkhorn normalisation of the soft group assignments (paper Sec. 2 "Learned grouping"):
// Q = exp(S / tau), then N times "divide each column by its sum over the tokens, divide each row by its sum over
// the groups".
//
// Every iterate has the form Q = diag(r) exp(S / tau) diag(c).  A column division replaces c_g by
// 1 / sum_i r_i E_ig and a row division replaces r_i by 1 / sum_g E_ig c_g, so one pass over the scores per
// iteration is enough: with the current column offsets a token computes its row offset (a log-sum-exp over K
// values), its normalised row Q_i (every entry in (0, 1]) and adds that row into the column sums that give the next
// column offsets.  Offsets are kept as logarithms, so nothing overflows at a small temperature; the very first
// column sum is taken relative to the column maximum.  Column sums are accumulated in fp64.
//
// The score matrix (n x K fp32, a few MB) stays in L2 between the passes; a pass is one small launch, and the
// N + 2 launches, not bandwidth, set the time.
#include "common.cuh"

namespace focus {

constexpr int SK_THREADS = 256;
constexpr int SK_MAX_BLOCKS = 148 * 8;

// order-preserving map of a float onto unsigned integers (0 sorts below every float)
__device__ __forceinline__ uint32_t ordered_of(float f) {
    const uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float float_of_ordered(uint32_t o) {
    return __uint_as_float((o & 0x80000000u) ? (o & 0x7fffffffu) : ~o);
}

// workspace of one sequence: double T[iters + 1][32] (column sums of pass 0, 1, ...), then uint32 M[32] (column maxima)
__host__ __device__ inline size_t sk_seq_bytes(int iters) { return (size_t)(iters + 1) * 32 * sizeof(double) + 32 * sizeof(uint32_t); }

template <int KMAX>
__device__ __forceinline__ void load_row(const float* __restrict__ S, size_t tok, float (&x)[KMAX]) {
    const float4* p = reinterpret_cast<const float4*>(S + tok * KMAX);
#pragma unroll
    for (int c = 0; c < KMAX / 4; ++c) {
        const float4 v = __ldg(p + c);
        x[4 * c] = v.x; x[4 * c + 1] = v.y; x[4 * c + 2] = v.z; x[4 * c + 3] = v.w;
    }
}

template <int KMAX>
__global__ void __launch_bounds__(SK_THREADS)
sinkhorn_colmax_kernel(const float* __restrict__ S, int n, int K, int iters, unsigned char* __restrict__ ws) {
    const int b = blockIdx.y;
    uint32_t* M = reinterpret_cast<uint32_t*>(ws + (size_t)b * sk_seq_bytes(iters) + (size_t)(iters + 1) * 32 * sizeof(double));
    const float* Sb = S + (size_t)b * n * KMAX;
    float mx[KMAX];
#pragma unroll
    for (int g = 0; g < KMAX; ++g) mx[g] = -INFINITY;
    for (int tok = blockIdx.x * SK_THREADS + threadIdx.x; tok < n; tok += gridDim.x * SK_THREADS) {
        float x[KMAX];
        load_row<KMAX>(Sb, (size_t)tok, x);
#pragma unroll
        for (int g = 0; g < KMAX; ++g) mx[g] = fmaxf(mx[g], x[g]);
    }
#pragma unroll
    for (int g = 0; g < KMAX; ++g) {
        float m = mx[g];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if ((threadIdx.x & 31) == 0 && g < K && m > -INFINITY) atomicMax(M + g, ordered_of(m));
    }
}

// MODE 0: column sums of exp((S - M) / tau).  MODE 1: a row division followed by the next column sums.
// MODE 2: the last row division; writes the assignments.
template <int KMAX, int MODE>
__global__ void __launch_bounds__(SK_THREADS)
sinkhorn_pass_kernel(const float* __restrict__ S, int n, int K, int iters, int pass, float inv_tau,
                     unsigned char* __restrict__ ws, float* __restrict__ out) {
    __shared__ double red[SK_THREADS / 32][KMAX];
    __shared__ float colmax_s[KMAX], voff_s[KMAX];
    const int b = blockIdx.y;
    unsigned char* wsb = ws + (size_t)b * sk_seq_bytes(iters);
    double* T = reinterpret_cast<double*>(wsb);
    const uint32_t* M = reinterpret_cast<const uint32_t*>(wsb + (size_t)(iters + 1) * 32 * sizeof(double));
    const float* Sb = S + (size_t)b * n * KMAX;
    if (threadIdx.x < KMAX) {
        const int g = threadIdx.x;
        float cm = 0.f, v = 0.f;
        if (g < K) {
            cm = float_of_ordered(M[g]);
            // column offset after `pass` column divisions, relative to the column maximum:
            // -log of the first column sum, then minus the log of every later one
            double acc = 0.0;
            for (int m = 0; m < pass; ++m) acc -= log(T[(size_t)m * 32 + g]);
            v = (float)acc;
        }
        colmax_s[g] = cm;
        voff_s[g] = v;
    }
    __syncthreads();
    float tsum[KMAX];
#pragma unroll
    for (int g = 0; g < KMAX; ++g) tsum[g] = 0.f;
    for (int tok = blockIdx.x * SK_THREADS + threadIdx.x; tok < n; tok += gridDim.x * SK_THREADS) {
        float x[KMAX];
        load_row<KMAX>(Sb, (size_t)tok, x);
        if (MODE == 0) {
#pragma unroll
            for (int g = 0; g < KMAX; ++g)
                if (g < K) tsum[g] += expf((x[g] - colmax_s[g]) * inv_tau);
        } else {
            float mx = -INFINITY;
#pragma unroll
            for (int g = 0; g < KMAX; ++g) {
                x[g] = (x[g] - colmax_s[g]) * inv_tau + voff_s[g];
                if (g < K) mx = fmaxf(mx, x[g]);
            }
            float se = 0.f;
#pragma unroll
            for (int g = 0; g < KMAX; ++g) {
                x[g] = g < K ? expf(x[g] - mx) : 0.f;
                se += x[g];
            }
            const float inv = 1.f / se;
#pragma unroll
            for (int g = 0; g < KMAX; ++g) x[g] *= inv;
            if (MODE == 1) {
#pragma unroll
                for (int g = 0; g < KMAX; ++g) tsum[g] += x[g];
            } else {
                float4* o = reinterpret_cast<float4*>(out + ((size_t)b * n + tok) * KMAX);
#pragma unroll
                for (int c = 0; c < KMAX / 4; ++c) o[c] = make_float4(x[4 * c], x[4 * c + 1], x[4 * c + 2], x[4 * c + 3]);
            }
        }
    }
    if (MODE != 2) {
#pragma unroll
        for (int g = 0; g < KMAX; ++g) {
            float s = tsum[g];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5][g] = (double)s;
        }
        __syncthreads();
        if (threadIdx.x < K) {
            double s = 0.0;
            for (int w = 0; w < SK_THREADS / 32; ++w) s += red[w][threadIdx.x];
            atomicAdd(T + (size_t)pass * 32 + threadIdx.x, s);
        }
    }
}

size_t sinkhorn_workspace_bytes(const focus_shape* s, int iters) { return (size_t)s->batch * sk_seq_bytes(iters); }

template <int KMAX>
static int launch_sk(const focus_shape* s, const float* S, float tau, int iters, unsigned char* ws, float* out, cudaStream_t st) {
    const int n = s->n, K = s->K;
    int nblk = cdiv(n, SK_THREADS);
    if (nblk > SK_MAX_BLOCKS) nblk = SK_MAX_BLOCKS;
    const dim3 grid(nblk, s->batch);
    const float inv_tau = 1.f / tau;
    int rc = check_cuda(cudaMemsetAsync(ws, 0, sinkhorn_workspace_bytes(s, iters), st), "cudaMemsetAsync(sinkhorn workspace)");
    if (rc) return rc;
    sinkhorn_colmax_kernel<KMAX><<<grid, SK_THREADS, 0, st>>>(S, n, K, iters, ws);
    sinkhorn_pass_kernel<KMAX, 0><<<grid, SK_THREADS, 0, st>>>(S, n, K, iters, 0, inv_tau, ws, nullptr);
    for (int pass = 1; pass < iters; ++pass)
        sinkhorn_pass_kernel<KMAX, 1><<<grid, SK_THREADS, 0, st>>>(S, n, K, iters, pass, inv_tau, ws, nullptr);
    sinkhorn_pass_kernel<KMAX, 2><<<grid, SK_THREADS, 0, st>>>(S, n, K, iters, iters, inv_tau, ws, out);
    return check_cuda(cudaGetLastError(), "sinkhorn kernel launch");
}

int launch_sinkhorn(const focus_shape* s, const float* S, float tau, int iters, void* ws, float* out, cudaStream_t st) {
    unsigned char* w = reinterpret_cast<unsigned char*>(ws);
    if (s->K <= 4) return launch_sk<4>(s, S, tau, iters, w, out, st);
    if (s->K <= 8) return launch_sk<8>(s, S, tau, iters, w, out, st);
    if (s->K <= 16) return launch_sk<16>(s, S, tau, iters, w, out, st);
    return launch_sk<32>(s, S, tau, iters, w, out, st);
}

// ---- backward: d loss / d S from d loss / d g (paper Sec. 2 "Learned grouping": the Sinkhorn steps are differentiated
// through, step by step in reverse).  With X_0 = exp(S / tau) and per iteration t: c_t = column sums of X_t,
// Y_t = X_t / c_t, r_t = row sums of Y_t, Z_t = Y_t / r_t = X_{t+1}, a division by a sum along an axis has the
// derivative dX = (dZ - sum(dZ * Z)) / sum(X) along that axis.  Every X_t row follows from its score row and the
// column sums the forward passes leave in the workspace, so nothing but those sums is taped: pass t of the
// backward recomputes the row's X_t, applies the column step left over from iteration t + 1 (its column sums are
// complete by then), then the row step of iteration t, and adds the row into the column sums iteration t needs.
// For t = 0 the division by r_0 is left to the last kernel, which needs only Z_0 = Y_0 / r_0 and Y_0: r_0 itself
// underflows for a row whose scores all lie far below the column maxima.
//
// B = double [iters][32] per sequence: column sums of d * Y_t.
template <int KMAX>
__global__ void __launch_bounds__(SK_THREADS)
sinkhorn_bwd_pass_kernel(const float* __restrict__ S, int n, int K, int iters, int t, float inv_tau,
                         const unsigned char* __restrict__ ws, double* __restrict__ B, const float* __restrict__ d_in,
                         float* __restrict__ d_out) {
    __shared__ double red[SK_THREADS / 32][KMAX];
    __shared__ float colmax_s[KMAX], voff_s[KMAX], pend_sub_s[KMAX], pend_inv_s[KMAX], ct_s[KMAX];
    const int b = blockIdx.y;
    const unsigned char* wsb = ws + (size_t)b * sk_seq_bytes(iters);
    const double* T = reinterpret_cast<const double*>(wsb);
    const uint32_t* M = reinterpret_cast<const uint32_t*>(wsb + (size_t)(iters + 1) * 32 * sizeof(double));
    double* Bb = B + (size_t)b * iters * 32;
    const float* Sb = S + (size_t)b * n * KMAX;
    const bool pending = t + 1 < iters;            // the column step of iteration t + 1 has not been applied yet
    if (threadIdx.x < KMAX) {
        const int g = threadIdx.x;
        float cm = 0.f, v = 0.f, ps = 0.f, pi = 0.f;
        if (g < K) {
            cm = float_of_ordered(M[g]);
            // log Y_t = (S - M) / tau - sum_{m <= t} log T[m]  (+ the row's own offset when t >= 1)
            double acc = 0.0;
            for (int m = 0; m <= t; ++m) acc -= log(T[(size_t)m * 32 + g]);
            v = (float)acc;
            if (pending) {
                ps = (float)Bb[(size_t)(t + 1) * 32 + g];
                pi = (float)(1.0 / T[(size_t)(t + 1) * 32 + g]);
            }
        }
        colmax_s[g] = cm; voff_s[g] = v; pend_sub_s[g] = ps; pend_inv_s[g] = pi;
        ct_s[g] = (g < K && t >= 1) ? (float)T[(size_t)t * 32 + g] : 0.f;
    }
    __syncthreads();
    float tsum[KMAX];
#pragma unroll
    for (int g = 0; g < KMAX; ++g) tsum[g] = 0.f;
    for (int tok = blockIdx.x * SK_THREADS + threadIdx.x; tok < n; tok += gridDim.x * SK_THREADS) {
        float x[KMAX], d[KMAX];
        load_row<KMAX>(Sb, (size_t)tok, x);
        load_row<KMAX>(d_in + (size_t)b * n * KMAX, (size_t)tok, d);
        // Z_t = softmax over the groups of log Y_t up to the row's offset; r_t = the sum that normalises it
        float mx = -INFINITY;
#pragma unroll
        for (int g = 0; g < KMAX; ++g) {
            x[g] = (x[g] - colmax_s[g]) * inv_tau + voff_s[g];
            if (g < K) mx = fmaxf(mx, x[g]);
        }
        float se = 0.f;
#pragma unroll
        for (int g = 0; g < KMAX; ++g) {
            x[g] = g < K ? expf(x[g] - mx) : 0.f;
            se += x[g];
        }
        const float inv = 1.f / se;
        float dot = 0.f;
#pragma unroll
        for (int g = 0; g < KMAX; ++g) {
            x[g] *= inv;                                           // Z_t
            d[g] = g < K ? (pending ? (d[g] - pend_sub_s[g]) * pend_inv_s[g] : d[g]) : 0.f;
            dot = fmaf(d[g], x[g], dot);
        }
        // 1 / r_t for t >= 1: the row of X_t = Z_{t-1} sums to one, Y_t = X_t / c_t = Z_t r_t, so
        // sum_g Y_t,g c_t,g = 1 = r_t sum_g Z_t,g c_t,g
        float rinv = 1.f;
        if (t >= 1) {
            float zc = 0.f;
#pragma unroll
            for (int g = 0; g < KMAX; ++g) zc = fmaf(x[g], ct_s[g], zc);
            rinv = zc;
        }
#pragma unroll
        for (int g = 0; g < KMAX; ++g) {
            const float e = d[g] - dot;
            tsum[g] += e * x[g];                                   // (d - dot) / r_t * Y_t = (d - dot) * Z_t
            d[g] = g < K ? e * rinv : 0.f;                         // t = 0: left undivided
        }
        float4* o = reinterpret_cast<float4*>(d_out + ((size_t)b * n + tok) * KMAX);
#pragma unroll
        for (int c = 0; c < KMAX / 4; ++c) o[c] = make_float4(d[4 * c], d[4 * c + 1], d[4 * c + 2], d[4 * c + 3]);
    }
#pragma unroll
    for (int g = 0; g < KMAX; ++g) {
        float s = tsum[g];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5][g] = (double)s;
    }
    __syncthreads();
    if (threadIdx.x < K) {
        double s = 0.0;
        for (int w = 0; w < SK_THREADS / 32; ++w) s += red[w][threadIdx.x];
        atomicAdd(Bb + (size_t)t * 32 + threadIdx.x, s);
    }
}

// dS = ((d - dot_0) * Z_0 - B_0 * Y_0) / tau, with e = d - dot_0 as pass 0 left it
template <int KMAX>
__global__ void __launch_bounds__(SK_THREADS)
sinkhorn_bwd_last_kernel(const float* __restrict__ S, int n, int K, int iters, float inv_tau,
                         const unsigned char* __restrict__ ws, const double* __restrict__ B, const float* __restrict__ d_in,
                         float* __restrict__ d_out) {
    __shared__ float colmax_s[KMAX], voff_s[KMAX], b0_s[KMAX];
    const int b = blockIdx.y;
    const unsigned char* wsb = ws + (size_t)b * sk_seq_bytes(iters);
    const double* T = reinterpret_cast<const double*>(wsb);
    const uint32_t* M = reinterpret_cast<const uint32_t*>(wsb + (size_t)(iters + 1) * 32 * sizeof(double));
    const float* Sb = S + (size_t)b * n * KMAX;
    if (threadIdx.x < KMAX) {
        const int g = threadIdx.x;
        colmax_s[g] = g < K ? float_of_ordered(M[g]) : 0.f;
        voff_s[g] = g < K ? (float)(-log(T[g])) : 0.f;
        b0_s[g] = g < K ? (float)B[(size_t)b * iters * 32 + g] : 0.f;
    }
    __syncthreads();
    for (int tok = blockIdx.x * SK_THREADS + threadIdx.x; tok < n; tok += gridDim.x * SK_THREADS) {
        float x[KMAX], e[KMAX];
        load_row<KMAX>(Sb, (size_t)tok, x);
        load_row<KMAX>(d_in + (size_t)b * n * KMAX, (size_t)tok, e);
        float mx = -INFINITY;
#pragma unroll
        for (int g = 0; g < KMAX; ++g) {
            x[g] = (x[g] - colmax_s[g]) * inv_tau + voff_s[g];     // log Y_0
            if (g < K) mx = fmaxf(mx, x[g]);
        }
        float se = 0.f, y[KMAX];
#pragma unroll
        for (int g = 0; g < KMAX; ++g) {
            y[g] = g < K ? expf(x[g]) : 0.f;                       // Y_0 (may underflow to 0: then its term vanishes)
            x[g] = g < K ? expf(x[g] - mx) : 0.f;
            se += x[g];
        }
        const float inv = 1.f / se;
#pragma unroll
        for (int g = 0; g < KMAX; ++g) e[g] = g < K ? (e[g] * (x[g] * inv) - b0_s[g] * y[g]) * inv_tau : 0.f;
        float4* o = reinterpret_cast<float4*>(d_out + ((size_t)b * n + tok) * KMAX);
#pragma unroll
        for (int c = 0; c < KMAX / 4; ++c) o[c] = make_float4(e[4 * c], e[4 * c + 1], e[4 * c + 2], e[4 * c + 3]);
    }
}

size_t sinkhorn_bwd_workspace_bytes(const focus_shape* s, int iters) {
    return (size_t)s->batch * (sk_seq_bytes(iters) + (size_t)iters * 32 * sizeof(double));
}

template <int KMAX>
static int launch_sk_bwd(const focus_shape* s, const float* S, float tau, int iters, unsigned char* ws, const float* dG, float* dS,
                         cudaStream_t st) {
    const int n = s->n, K = s->K;
    int nblk = cdiv(n, SK_THREADS);
    if (nblk > SK_MAX_BLOCKS) nblk = SK_MAX_BLOCKS;
    const dim3 grid(nblk, s->batch);
    const float inv_tau = 1.f / tau;
    int rc = check_cuda(cudaMemsetAsync(ws, 0, sinkhorn_bwd_workspace_bytes(s, iters), st), "cudaMemsetAsync(sinkhorn workspace)");
    if (rc) return rc;
    double* B = reinterpret_cast<double*>(ws + (size_t)s->batch * sk_seq_bytes(iters));
    // the forward's column sums again (no assignments written)
    sinkhorn_colmax_kernel<KMAX><<<grid, SK_THREADS, 0, st>>>(S, n, K, iters, ws);
    sinkhorn_pass_kernel<KMAX, 0><<<grid, SK_THREADS, 0, st>>>(S, n, K, iters, 0, inv_tau, ws, nullptr);
    for (int pass = 1; pass < iters; ++pass)
        sinkhorn_pass_kernel<KMAX, 1><<<grid, SK_THREADS, 0, st>>>(S, n, K, iters, pass, inv_tau, ws, nullptr);
    for (int t = iters - 1; t >= 0; --t)
        sinkhorn_bwd_pass_kernel<KMAX><<<grid, SK_THREADS, 0, st>>>(S, n, K, iters, t, inv_tau, ws, B, t == iters - 1 ? dG : dS, dS);
    sinkhorn_bwd_last_kernel<KMAX><<<grid, SK_THREADS, 0, st>>>(S, n, K, iters, inv_tau, ws, B, dS, dS);
    return check_cuda(cudaGetLastError(), "sinkhorn backward kernel launch");
}

int launch_sinkhorn_bwd(const focus_shape* s, const float* S, float tau, int iters, void* ws, const float* dG, float* dS,
                        cudaStream_t st) {
    unsigned char* w = reinterpret_cast<unsigned char*>(ws);
    if (s->K <= 4) return launch_sk_bwd<4>(s, S, tau, iters, w, dG, dS, st);
    if (s->K <= 8) return launch_sk_bwd<8>(s, S, tau, iters, w, dG, dS, st);
    if (s->K <= 16) return launch_sk_bwd<16>(s, S, tau, iters, w, dG, dS, st);
    return launch_sk_bwd<32>(s, S, tau, iters, w, dG, dS, st);
}

}  // namespace focus
