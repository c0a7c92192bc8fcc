// C-ABI entry points: argument validation, workspace layout, dispatch.  No kernels here.
#include "common.cuh"

#include <stdlib.h>
#include <string.h>

namespace focus {

static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
}

int fail(int status, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return status;
}

int check_cuda(cudaError_t e, const char* what) {
    if (e == cudaSuccess) return FOCUS_OK;
    return fail(FOCUS_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

int validate_shape(const focus_shape* s) {
    if (!s) return fail(FOCUS_ERR_INVALID_ARG, "shape is NULL");
    if (s->batch < 1 || s->Hq < 1 || s->Hkv < 1 || s->n < 1)
        return fail(FOCUS_ERR_INVALID_ARG, "batch, Hq, Hkv and n must be >= 1");
    if (s->Hq % s->Hkv) return fail(FOCUS_ERR_INVALID_ARG, "Hq (%d) is not a multiple of Hkv (%d)", s->Hq, s->Hkv);
    if (s->K < 1 || s->K > 32) return fail(FOCUS_ERR_INVALID_ARG, "K (%d) outside [1,32]", s->K);
    if (s->topk < 1 || s->topk > s->K) return fail(FOCUS_ERR_INVALID_ARG, "topk (%d) outside [1,K]", s->topk);
    if (s->window < 0) return fail(FOCUS_ERR_INVALID_ARG, "window must be >= 0");
    if (!(s->scale >= 0.f) || !(s->softcap >= 0.f))
        return fail(FOCUS_ERR_INVALID_ARG, "scale and softcap must be >= 0 (0 = default / off)");
    if (s->D != 64 && s->D != 128 && s->D != 256)
        return fail(FOCUS_ERR_UNSUPPORTED, "D (%d) must be 64, 128 or 256", s->D);
    if ((long long)s->batch * s->Hq > (1 << 20)) return fail(FOCUS_ERR_INVALID_ARG, "batch*Hq too large");
    if (s->n > (1 << 30)) return fail(FOCUS_ERR_INVALID_ARG, "n too large");
    return FOCUS_OK;
}

int validate_tensor(const char* name, const focus_tensor& t, bool tma, int batch) {
    if (!t.ptr) return fail(FOCUS_ERR_INVALID_ARG, "%s.ptr is NULL", name);
    if (t.stride_n < 1 || t.stride_h < 1 || t.stride_b < 0)
        return fail(FOCUS_ERR_INVALID_ARG, "%s has a non-positive stride", name);
    // a batch stride of 0 is accepted as "unused" for a single sequence only: with batch > 1 it would
    // alias every sequence onto the first one
    if (batch > 1 && t.stride_b < 1)
        return fail(FOCUS_ERR_INVALID_ARG, "%s.stride_b must be positive when batch > 1", name);
    if (tma) {
        if ((uintptr_t)t.ptr % 16) return fail(FOCUS_ERR_INVALID_ARG, "%s.ptr is not 16-byte aligned", name);
        if (t.stride_n % 8 || t.stride_h % 8 || t.stride_b % 8)
            return fail(FOCUS_ERR_INVALID_ARG, "%s strides must be multiples of 8 elements", name);
    }
    return FOCUS_OK;
}

int require_sm100() {
    int dev = 0, major = 0;
    int rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
    if (rc) return rc;
    rc = check_cuda(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev), "cudaDeviceGetAttribute");
    if (rc) return rc;
    if (major != 10) return fail(FOCUS_ERR_ARCH, "device compute capability %d.x is not 10.x (B200)", major);
    return FOCUS_OK;
}

// C(a, b) as a double (a <= 32)
static double binom(int a, int b) {
    if (b < 0 || b > a) return 0.0;
    double r = 1.0;
    for (int j = 0; j < b; ++j) r = r * (a - j) / (j + 1);
    return r;
}

// FOCUS_LAYOUT_AUTO: a function of the shape alone, so that every entry point resolves it alike
static int choose_layout(const focus_shape* s) {
    const double classes = binom(s->K, s->topk);
    if (classes > (double)FOCUS_MAX_CLASSES + 0.5) return FOCUS_LAYOUT_ORIGINAL;
    const double dropped = binom(s->K - s->topk, s->topk) / classes;      // far pairs without a shared group, uniform memberships
    // Which of the two class-sorted layouts.  Key tiles a block of 256 sorted queries visits for its window alone: its
    // rows span about 256 * classes positions, so the window of the block covers (256 * classes + w) / classes keys of
    // every class that shares no group with it.  The separate window pass in token order reads w + 256 keys once per
    // 256 rows, plus what a second pass costs per block whatever its length (query load, pipeline fill, fp32 partial
    // results, merge): about six key tiles' worth, measured.  The pass is taken when it saves a quarter or more.
    const double apart = binom(s->K - s->topk, s->topk);                 // classes without a shared group
    const double in_sorted = apart * ((256.0 * classes + s->window) / classes / 128.0 + 1.0);
    const double in_order = (s->window + 256.0) / 128.0 + 7.0;
    const int sorted = in_sorted > 1.25 * in_order ? FOCUS_LAYOUT_SORTED_LOCAL : FOCUS_LAYOUT_CLASS_SORTED;
    // long enough for the fixed costs of sorting: 2048 tokens per class, 1024 when the window has its own pass
    const double per_class = sorted == FOCUS_LAYOUT_SORTED_LOCAL ? 1024.0 : 2048.0;
    const double min_n = classes * per_class > 16384.0 ? classes * per_class : 16384.0;
    if ((double)s->n < min_n) return FOCUS_LAYOUT_ORIGINAL;
    if (dropped >= 0.5 || (s->n >= 65536 && dropped >= 0.15)) return sorted;
    return FOCUS_LAYOUT_ORIGINAL;
}

static int layout_of(const focus_shape* s, int layout, focus_tiles_layout* L) {
    int rc = validate_shape(s);
    if (rc) return rc;
    if (!L) return fail(FOCUS_ERR_INVALID_ARG, "out is NULL");
    if (layout == FOCUS_LAYOUT_AUTO) layout = choose_layout(s);
    if (layout != FOCUS_LAYOUT_ORIGINAL && !layout_is_sorted(layout))
        return fail(FOCUS_ERR_INVALID_ARG,
                    "layout must be 0 (original), 1 (class-sorted), 2 (chosen by the library), 3 (class-sorted + window pass) "
                    "or 4 (group-major keys + window pass)");
    if (layout == FOCUS_LAYOUT_GROUP_MAJOR && group_major_capacity(s) > (1ll << 30))
        return fail(FOCUS_ERR_UNSUPPORTED, "group-major layout: n * topk is too large");
    memset(L, 0, sizeof *L);
    const size_t HQ = (size_t)s->batch * s->Hq, HK = (size_t)s->batch * s->Hkv;
    L->layout = layout;
    L->nqt = cdiv(s->n, FOCUS_TILE_M);
    L->nkt = cdiv(s->n, FOCUS_TILE_N);
    L->nkw = cdiv(L->nkt, 32);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L->counters = take(8 * sizeof(uint64_t));
    L->orq = take(HQ * L->nqt * 4);
    L->andq = take(HQ * L->nqt * 4);
    L->ork = take(HK * L->nkt * 4);
    L->andk = take(HK * L->nkt * 4);
    L->gbits = take(HK * L->nkt * (size_t)s->K * 4 * 4);
    L->live = take(HQ * L->nqt * (size_t)L->nkw * 4);
    L->live_cnt = take(HQ * L->nqt * 4);
    L->kany = take(HK * (size_t)s->K * L->nkw * 4);
    L->kall = take(HK * (size_t)s->K * L->nkw * 4);
    if (layout_is_sorted(layout)) {
        L->nqp = sorted_capacity(s->n);
        L->nkp = layout == FOCUS_LAYOUT_GROUP_MAJOR ? (int)group_major_capacity(s) : sorted_capacity(s->n);
        L->ncls_q = take(HQ * 4);
        L->ncls_k = take(HK * 4);
        L->cls_q = take(HQ * FOCUS_MAX_CLASSES * 4);
        L->cls_k = take(HK * FOCUS_MAX_CLASSES * 4);
        L->cnt_q = take(HQ * FOCUS_MAX_CLASSES * 4);
        L->cnt_k = take(HK * FOCUS_MAX_CLASSES * 4);
        L->seg_q = take(HQ * (FOCUS_MAX_CLASSES + 1) * 4);
        L->seg_k = take(HK * (FOCUS_MAX_CLASSES + 1) * 4);
        L->perm_q = take(HQ * (size_t)L->nqp * 4);
        L->perm_k = take(HK * (size_t)L->nkp * 4);
        L->qrange = take(HQ * (size_t)(L->nqp / 256) * FOCUS_MAX_CLASSES * 2 * 4);
        L->order = take(HQ * (size_t)(L->nqp / 256) * 2 * 4);
        if (layout == FOCUS_LAYOUT_GROUP_MAJOR) L->gbits_s = take(HK * (size_t)(L->nkp / 128) * (size_t)s->K * 4 * 4);
        L->qs = take(HQ * (size_t)L->nqp * s->D * 2);
        L->ks = take(HK * (size_t)L->nkp * s->D * 2);
        L->vs = take(HK * (size_t)L->nkp * s->D * 2);
        L->scratch = take(sorted_scratch_bytes(s));
    }
    if (layout_has_window_pass(layout)) {
        L->o_sorted = take(HQ * (size_t)s->n * s->D * 4);
        L->o_local = take(HQ * (size_t)s->n * s->D * 4);
        L->lse_local = take(HQ * (size_t)s->n * 4);
    }
    L->total_bytes = off;
    return FOCUS_OK;
}

}  // namespace focus

using namespace focus;

extern "C" {

int focus_version(void) { return 100; }

const char* focus_status_string(int status) {
    switch (status) {
        case FOCUS_OK: return "ok";
        case FOCUS_ERR_INVALID_ARG: return "invalid argument";
        case FOCUS_ERR_UNSUPPORTED: return "unsupported configuration";
        case FOCUS_ERR_CAPACITY: return "workspace too small";
        case FOCUS_ERR_ARCH: return "device is not sm_100";
        case FOCUS_ERR_CUDA: return "CUDA error";
        default: return "unknown status";
    }
}

const char* focus_last_error(void) { return g_err; }

int focus_tiles_layout_of(const focus_shape* shape, int32_t layout, focus_tiles_layout* out) {
    return layout_of(shape, layout, out);
}

size_t focus_tiles_workspace_bytes(const focus_shape* shape, int32_t layout) {
    focus_tiles_layout L;
    if (layout_of(shape, layout, &L)) return 0;
    return L.total_bytes;
}

int focus_assign(const focus_shape* shape, focus_tensor x, int32_t H, const float* centroids, uint32_t* masks_out,
                 unsigned long long* near_ties, float near_tie_eps, void* stream) {
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (H != shape->Hq && H != shape->Hkv) return fail(FOCUS_ERR_INVALID_ARG, "H (%d) must be Hq or Hkv", H);
    if ((rc = validate_tensor("x", x, false, shape->batch))) return rc;
    if ((uintptr_t)x.ptr % 16 || x.stride_n % 8 || x.stride_h % 8 || x.stride_b % 8)
        return fail(FOCUS_ERR_INVALID_ARG, "x must be 16-byte aligned with strides that are multiples of 8 elements");
    if (!centroids || !masks_out) return fail(FOCUS_ERR_INVALID_ARG, "centroids or masks_out is NULL");
    if ((rc = require_sm100())) return rc;
    return launch_assign(shape, x, H, centroids, masks_out, near_ties, near_tie_eps, (cudaStream_t)stream);
}

int focus_assign_hidden(const focus_shape* shape, const void* h, int64_t stride_b, int64_t stride_n, int32_t d_model,
                        int32_t d_g, const float* Wg, const float* C, const float* bias, float* folded, uint32_t* mq_out,
                        uint32_t* mk_out, unsigned long long* near_ties, float near_tie_eps, void* stream) {
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (!h || !Wg || !C || !folded) return fail(FOCUS_ERR_INVALID_ARG, "h, Wg, C or folded is NULL");
    if (!mq_out && !mk_out) return fail(FOCUS_ERR_INVALID_ARG, "mq_out and mk_out are both NULL");
    if (d_model < 8 || d_model % 8 || d_g < 1) return fail(FOCUS_ERR_INVALID_ARG, "d_model must be a positive multiple of 8 and d_g >= 1");
    if ((uintptr_t)h % 16 || (uintptr_t)folded % 16 || stride_n % 8 || stride_b % 8 || stride_n < d_model)
        return fail(FOCUS_ERR_INVALID_ARG, "h and folded must be 16-byte aligned, strides multiples of 8 elements, stride_n >= d_model");
    if ((rc = require_sm100())) return rc;
    return launch_assign_hidden(shape, h, stride_b, stride_n, d_model, d_g, Wg, C, bias, folded, mq_out, mk_out, near_ties,
                                near_tie_eps, nullptr, (cudaStream_t)stream);
}

int32_t focus_soft_ld(int32_t K) {
    if (K < 1 || K > 32) return 0;
    return K <= 4 ? 4 : (K <= 8 ? 8 : (K <= 16 ? 16 : 32));
}

int focus_router_scores(const focus_shape* shape, const void* h, int64_t stride_b, int64_t stride_n, int32_t d_model,
                        int32_t d_g, const float* Wg, const float* C, float* folded, float* scores_out, void* stream) {
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (!h || !Wg || !C || !folded || !scores_out) return fail(FOCUS_ERR_INVALID_ARG, "h, Wg, C, folded or scores_out is NULL");
    if (d_model < 8 || d_model % 8 || d_g < 1) return fail(FOCUS_ERR_INVALID_ARG, "d_model must be a positive multiple of 8 and d_g >= 1");
    if ((uintptr_t)h % 16 || (uintptr_t)folded % 16 || (uintptr_t)scores_out % 16 || stride_n % 8 || stride_b % 8 || stride_n < d_model)
        return fail(FOCUS_ERR_INVALID_ARG,
                    "h, folded and scores_out must be 16-byte aligned, strides multiples of 8 elements, stride_n >= d_model");
    if ((rc = require_sm100())) return rc;
    return launch_assign_hidden(shape, h, stride_b, stride_n, d_model, d_g, Wg, C, nullptr, folded, nullptr, nullptr, nullptr, 0.f,
                                scores_out, (cudaStream_t)stream);
}

size_t focus_sinkhorn_workspace_bytes(const focus_shape* shape, int32_t iters) {
    if (validate_shape(shape) || iters < 1) return 0;
    return sinkhorn_workspace_bytes(shape, iters);
}

int focus_sinkhorn(const focus_shape* shape, const float* scores, float tau, int32_t iters, void* ws, size_t ws_bytes,
                   float* g_out, void* stream) {
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (!scores || !ws || !g_out) return fail(FOCUS_ERR_INVALID_ARG, "scores, ws or g_out is NULL");
    if (!(tau > 0.f) || iters < 1 || iters > 1000) return fail(FOCUS_ERR_INVALID_ARG, "tau must be positive and iters in [1, 1000]");
    if ((uintptr_t)scores % 16 || (uintptr_t)g_out % 16 || (uintptr_t)ws % 16)
        return fail(FOCUS_ERR_INVALID_ARG, "scores, g_out and ws must be 16-byte aligned");
    if (ws_bytes < sinkhorn_workspace_bytes(shape, iters))
        return fail(FOCUS_ERR_CAPACITY, "sinkhorn workspace has %zu bytes, %zu needed", ws_bytes, sinkhorn_workspace_bytes(shape, iters));
    if ((rc = require_sm100())) return rc;
    return launch_sinkhorn(shape, scores, tau, iters, ws, g_out, (cudaStream_t)stream);
}

size_t focus_sinkhorn_bwd_workspace_bytes(const focus_shape* shape, int32_t iters) {
    if (validate_shape(shape) || iters < 1) return 0;
    return sinkhorn_bwd_workspace_bytes(shape, iters);
}

int focus_sinkhorn_bwd(const focus_shape* shape, const float* scores, float tau, int32_t iters, void* ws, size_t ws_bytes,
                       const float* dg, float* dscores_out, void* stream) {
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (!scores || !ws || !dg || !dscores_out) return fail(FOCUS_ERR_INVALID_ARG, "scores, ws, dg or dscores_out is NULL");
    if (!(tau > 0.f) || iters < 1 || iters > 1000) return fail(FOCUS_ERR_INVALID_ARG, "tau must be positive and iters in [1, 1000]");
    if ((uintptr_t)scores % 16 || (uintptr_t)dg % 16 || (uintptr_t)dscores_out % 16 || (uintptr_t)ws % 16)
        return fail(FOCUS_ERR_INVALID_ARG, "scores, dg, dscores_out and ws must be 16-byte aligned");
    if (dscores_out == scores) return fail(FOCUS_ERR_INVALID_ARG, "dscores_out must not be the scores buffer (the scores are read by every pass)");
    if (ws_bytes < sinkhorn_bwd_workspace_bytes(shape, iters))
        return fail(FOCUS_ERR_CAPACITY, "sinkhorn backward workspace has %zu bytes, %zu needed", ws_bytes,
                    sinkhorn_bwd_workspace_bytes(shape, iters));
    if ((rc = require_sm100())) return rc;
    return launch_sinkhorn_bwd(shape, scores, tau, iters, ws, dg, dscores_out, (cudaStream_t)stream);
}

int focus_build_tiles(const focus_shape* shape, const uint32_t* mq, const uint32_t* mk, int32_t layout, void* ws,
                      size_t ws_bytes, void* stream) {
    focus_tiles_layout L;
    int rc = layout_of(shape, layout, &L);
    if (rc) return rc;
    if (!mq || !mk || !ws) return fail(FOCUS_ERR_INVALID_ARG, "mq, mk or ws is NULL");
    if ((uintptr_t)ws % 256) return fail(FOCUS_ERR_INVALID_ARG, "ws is not 256-byte aligned");
    if (ws_bytes < L.total_bytes)
        return fail(FOCUS_ERR_CAPACITY, "workspace has %zu bytes, %zu needed", ws_bytes, L.total_bytes);
    layout = L.layout;                     // FOCUS_LAYOUT_AUTO resolved
    if (layout == FOCUS_LAYOUT_CLASS_SORTED || layout == FOCUS_LAYOUT_SORTED_LOCAL) {
        // masks with exactly topk bits have C(K, topk) values; more than the class table holds is refused here,
        // other mask patterns with too many values are caught on the device (counters[4], then dev_status).
        // (Group-major keys need the table for the query side only: checked on the device.)
        double classes = 1.0;
        for (int j = 0; j < shape->topk; ++j) classes = classes * (shape->K - j) / (j + 1);
        if (classes > (double)FOCUS_MAX_CLASSES + 0.5)
            return fail(FOCUS_ERR_UNSUPPORTED, "class-sorted layout: C(K=%d, topk=%d) mask values exceed %d", shape->K,
                        shape->topk, FOCUS_MAX_CLASSES);
    }
    if ((rc = require_sm100())) return rc;
    return launch_build_tiles(shape, mq, mk, layout, L, (char*)ws, (cudaStream_t)stream);
}

size_t focus_decode_workspace_bytes(const focus_shape* shape) {
    if (validate_shape(shape)) return 0;
    return decode_workspace_bytes(shape);
}

int focus_decode_step(const focus_shape* shape, focus_tensor q, focus_tensor k, focus_tensor v, const uint32_t* mq_new,
                      const uint32_t* mk, focus_tensor o, float* lse, void* ws, size_t ws_bytes, void* stream) {
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (!q.ptr || !o.ptr || !mq_new || !mk || !lse || !ws) return fail(FOCUS_ERR_INVALID_ARG, "a pointer argument is NULL");
    if ((rc = validate_tensor("k", k, true, shape->batch)) || (rc = validate_tensor("v", v, true, shape->batch))) return rc;
    // the query vectors are read two elements at a time
    if ((uintptr_t)q.ptr % 4 || q.stride_h % 2 || q.stride_b % 2 || q.stride_h < 1 || o.stride_h < 1 || q.stride_b < 0 ||
        o.stride_b < 0)
        return fail(FOCUS_ERR_INVALID_ARG, "q must be 4-byte aligned with even, positive head strides (o: positive strides)");
    if (shape->batch > 1 && (q.stride_b < 1 || o.stride_b < 1))
        return fail(FOCUS_ERR_INVALID_ARG, "q.stride_b and o.stride_b must be positive when batch > 1");
    if ((uintptr_t)ws % 16) return fail(FOCUS_ERR_INVALID_ARG, "ws is not 16-byte aligned");
    if (ws_bytes < decode_workspace_bytes(shape))
        return fail(FOCUS_ERR_CAPACITY, "decode workspace has %zu bytes, %zu needed", ws_bytes, decode_workspace_bytes(shape));
    if ((rc = require_sm100())) return rc;
    const float scale = shape->scale > 0.f ? shape->scale : 1.0f / sqrtf((float)shape->D);
    return launch_decode(shape, q, k, v, mq_new, mk, o, lse, (float*)ws, scale, (cudaStream_t)stream);
}

int focus_count_kept(const focus_shape* shape, const uint32_t* mq, const void* tiles_ws,
                     unsigned long long* counts_out, void* stream) {
    focus_tiles_layout L;
    int rc = layout_of(shape, FOCUS_LAYOUT_ORIGINAL, &L);   // the summaries sit at the same offsets in both layouts
    if (rc) return rc;
    if (!mq || !tiles_ws || !counts_out) return fail(FOCUS_ERR_INVALID_ARG, "mq, tiles_ws or counts_out is NULL");
    if ((rc = require_sm100())) return rc;
    return launch_count_kept(shape, mq, L, (const char*)tiles_ws, counts_out, (cudaStream_t)stream);
}

int focus_attn_fwd(const focus_shape* shape, focus_tensor q, focus_tensor k, focus_tensor v, const uint32_t* mq,
                   const uint32_t* mk, const void* tiles_ws, int32_t layout, focus_tensor o, float* lse,
                   int32_t* dev_status, void* stream) {
    int rc = validate_shape(shape);
    if (rc) return rc;
    const int nb = shape->batch;
    if ((rc = validate_tensor("q", q, true, nb)) || (rc = validate_tensor("k", k, true, nb)) ||
        (rc = validate_tensor("v", v, true, nb)) || (rc = validate_tensor("o", o, true, nb)))
        return rc;
    if (!lse) return fail(FOCUS_ERR_INVALID_ARG, "lse is NULL");
    if (tiles_ws && (!mq || !mk)) return fail(FOCUS_ERR_INVALID_ARG, "mq/mk are required with a tiles workspace");
    AttnArgs a;
    a.s = *shape;
    a.q = q; a.k = k; a.v = v; a.o = o;
    a.mq = mq; a.mk = mk;
    a.ws = (const char*)tiles_ws;
    a.lse = lse;
    a.dev_status = dev_status;
    a.scale = shape->scale > 0.f ? shape->scale : 1.0f / sqrtf((float)shape->D);
    memset(&a.L, 0, sizeof a.L);
    if (tiles_ws && (rc = layout_of(shape, layout, &a.L))) return rc;
    // The sorted layouts can refuse on the device (more mask values in a head than the class table holds) and then leave
    // O / lse unwritten: the only way to learn of it is the status word, so it is required there.
    if (tiles_ws && a.L.layout != FOCUS_LAYOUT_ORIGINAL && !dev_status)
        return fail(FOCUS_ERR_INVALID_ARG, "dev_status is required with a sorted layout (it reports a refused class table)");
    if ((rc = require_sm100())) return rc;
    return launch_attn_sm100(a, (cudaStream_t)stream);
}

int focus_selftest_stalled_wait(const focus_shape* shape, focus_tensor q, focus_tensor k, focus_tensor v, focus_tensor o,
                                float* lse, unsigned long long wait_limit_ns, int32_t* dev_status, void* stream) {
    int rc = validate_shape(shape);
    if (rc) return rc;
    const int nb = shape->batch;
    if ((rc = validate_tensor("q", q, true, nb)) || (rc = validate_tensor("k", k, true, nb)) ||
        (rc = validate_tensor("v", v, true, nb)) || (rc = validate_tensor("o", o, true, nb)))
        return rc;
    if (!lse || !dev_status) return fail(FOCUS_ERR_INVALID_ARG, "lse or dev_status is NULL");
    if (wait_limit_ns < 1000ull || wait_limit_ns > 4000000000ull)
        return fail(FOCUS_ERR_INVALID_ARG, "wait_limit_ns must lie between 1 microsecond and 4 seconds");
    if (shape->n < 512) return fail(FOCUS_ERR_INVALID_ARG, "n must be at least 512 (the stalled stage is the fourth of an item)");
    if ((rc = require_sm100())) return rc;
    AttnArgs a;
    a.s = *shape;
    a.q = q; a.k = k; a.v = v; a.o = o;
    a.mq = nullptr; a.mk = nullptr;
    a.ws = nullptr;                        // dense causal walk
    a.lse = lse;
    a.dev_status = dev_status;
    a.scale = shape->scale > 0.f ? shape->scale : 1.0f / sqrtf((float)shape->D);
    memset(&a.L, 0, sizeof a.L);
    a.wait_limit_ns = wait_limit_ns;
    a.stall_at = 3;
    return launch_attn_sm100(a, (cudaStream_t)stream);
}

int focus_gate_attn_fwd(const focus_shape* shape, focus_tensor q, focus_tensor k, focus_tensor v, const float* g, float lambda,
                        focus_tensor o, float* lse, int32_t* dev_status, void* stream) {
    int rc = validate_shape(shape);
    if (rc) return rc;
    const int nb = shape->batch;
    if ((rc = validate_tensor("q", q, true, nb)) || (rc = validate_tensor("k", k, true, nb)) ||
        (rc = validate_tensor("v", v, true, nb)) || (rc = validate_tensor("o", o, true, nb)))
        return rc;
    if (!lse || !g) return fail(FOCUS_ERR_INVALID_ARG, "lse or g is NULL");
    if ((uintptr_t)g % 16) return fail(FOCUS_ERR_INVALID_ARG, "g is not 16-byte aligned");
    if (shape->softcap > 0.f) return fail(FOCUS_ERR_UNSUPPORTED, "the gated forward takes no softcap");
    if (shape->K > 32 || (shape->D == 256 && shape->K > 16))
        return fail(FOCUS_ERR_UNSUPPORTED, "the gated forward supports K <= 32 (K <= 16 at D = 256); K = %d", shape->K);
    if ((rc = require_sm100())) return rc;
    AttnArgs a;
    a.s = *shape;
    a.q = q; a.k = k; a.v = v; a.o = o;
    a.mq = nullptr; a.mk = nullptr;
    a.ws = nullptr;                        // every causal pair is computed
    a.lse = lse;
    a.dev_status = dev_status;
    a.scale = shape->scale > 0.f ? shape->scale : 1.0f / sqrtf((float)shape->D);
    memset(&a.L, 0, sizeof a.L);
    a.gate_g = g;
    a.gate_ld = focus_soft_ld(shape->K);
    a.gate_lambda = lambda;
    return launch_attn_sm100(a, (cudaStream_t)stream);
}

}  // extern "C"
