// Internal helpers shared by the translation units of libfocus_b200.so.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stdio.h>
#include <stdarg.h>

#include "focus.h"

namespace focus {

// thread-local error text behind focus_last_error()
void set_error(const char* fmt, ...);
int fail(int status, const char* fmt, ...);
int check_cuda(cudaError_t e, const char* what);

// shape validation shared by all entry points (0 or a negative status)
int validate_shape(const focus_shape* s);
// validation of a bf16 tensor argument; tma = also enforce 16-byte base alignment and stride % 8 == 0;
// batch > 1 requires a positive batch stride
int validate_tensor(const char* name, const focus_tensor& t, bool tma, int batch);
// current device must be compute capability 10.x
int require_sm100();

inline int cdiv(int a, int b) { return (a + b - 1) / b; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// layout-1 padded sorted length: room for every class segment to be rounded up to 256 slots
inline int sorted_capacity(int n) { return (int)align_up((size_t)n + (size_t)FOCUS_MAX_CLASSES * 255, 256); }
// group-major keys: every key once per group it belongs to (topk of them), every list padded to 128 slots
inline long long group_major_capacity(const focus_shape* s) {
    return (long long)align_up((size_t)s->n * (size_t)s->topk + (size_t)s->K * 127, 256);
}
inline bool layout_is_sorted(int layout) {
    return layout == FOCUS_LAYOUT_CLASS_SORTED || layout == FOCUS_LAYOUT_SORTED_LOCAL || layout == FOCUS_LAYOUT_GROUP_MAJOR;
}
inline bool layout_has_window_pass(int layout) { return layout == FOCUS_LAYOUT_SORTED_LOCAL || layout == FOCUS_LAYOUT_GROUP_MAJOR; }

// class-sorted layout, build-time scratch: per head a hash set of mask values (256 x 8 bytes), per head and
// chunk of 1024 tokens a histogram over classes, and per query block its number of key tiles
constexpr int SORT_CHUNK = 1024;
constexpr int SORT_HASH = 256;
inline size_t sorted_scratch_bytes(const focus_shape* s) {
    const size_t heads = (size_t)s->batch * (s->Hq + s->Hkv);
    const size_t nchunk = (size_t)cdiv(s->n, SORT_CHUNK);
    return align_up(heads * SORT_HASH * 8, 256) + align_up(heads * nchunk * FOCUS_MAX_CLASSES * 4, 256) +
           align_up((size_t)s->batch * s->Hq * (size_t)(sorted_capacity(s->n) / 256) * 4, 256);
}

// launchers implemented in the other translation units
int launch_assign(const focus_shape* s, const focus_tensor& x, int H, const float* centroids, uint32_t* masks,
                  unsigned long long* near_ties, float eps, cudaStream_t st);
int launch_assign_hidden(const focus_shape* s, const void* h, int64_t sb, int64_t sn, int d, int dg, const float* Wg,
                         const float* C, const float* bias, float* folded, uint32_t* mq, uint32_t* mk,
                         unsigned long long* near_ties, float eps, float* scores, cudaStream_t st);
size_t sinkhorn_workspace_bytes(const focus_shape* s, int iters);
int launch_sinkhorn(const focus_shape* s, const float* S, float tau, int iters, void* ws, float* out, cudaStream_t st);
size_t sinkhorn_bwd_workspace_bytes(const focus_shape* s, int iters);
int launch_sinkhorn_bwd(const focus_shape* s, const float* S, float tau, int iters, void* ws, const float* dG, float* dS,
                        cudaStream_t st);
size_t decode_workspace_bytes(const focus_shape* s);
int launch_decode(const focus_shape* s, const focus_tensor& q, const focus_tensor& k, const focus_tensor& v,
                  const uint32_t* mq_new, const uint32_t* mk, const focus_tensor& o, float* lse, float* part, float scale,
                  cudaStream_t st);
int launch_build_tiles(const focus_shape* s, const uint32_t* mq, const uint32_t* mk, int layout,
                       const focus_tiles_layout& L, char* ws, cudaStream_t st);
// class-sorted layout: copy the rows of t into the sorted order of the workspace (query or key side)
int launch_gather_sorted(const focus_shape* s, const focus_tensor& t, int H, bool query, const focus_tiles_layout& L,
                         const char* ws, char* dst, cudaStream_t st);
int launch_fill_f32(float* x, size_t count, float v, cudaStream_t st);
// FOCUS_LAYOUT_SORTED_LOCAL: the partial results of the class-sorted pass (o_sorted, lse) and of the window pass are joined into o, lse
int launch_merge_partials(const focus_shape* s, const focus_tensor& o, float* lse, const float* o_sorted, const float* o_local,
                          const float* lse_local, cudaStream_t st);
int launch_count_kept(const focus_shape* s, const uint32_t* mq, const focus_tiles_layout& L, const char* ws,
                      unsigned long long* out, cudaStream_t st);

struct AttnArgs {
    focus_shape s;
    focus_tensor q, k, v, o;
    const uint32_t* mq;
    const uint32_t* mk;
    const char* ws;           // nullptr = dense causal
    focus_tiles_layout L;     // valid when ws != nullptr
    float* lse;
    int32_t* dev_status;
    float scale;              // resolved logit scale
    float* o32 = nullptr;            // when set, O goes there in fp32, rows [batch*Hq][n][D], instead of to `o` (partial passes)
    bool local_pass = false;         // FOCUS_LAYOUT_SORTED_LOCAL: the window pass in token order (pairs without a shared group)
    const float* gate_g = nullptr;   // training-time soft gate: assignments [batch, n, gate_ld]; nullptr = no gate
    int gate_ld = 0;
    float gate_lambda = 0.f;
    unsigned long long wait_limit_ns = 4000000000ull;   // every wait inside the kernel gives up after this long
    long long stall_at = -1;         // diagnostic (focus_selftest_stalled_wait): a ring stage that is never filled
};
int launch_attn_sm100(const AttnArgs& a, cudaStream_t st);

}  // namespace focus
