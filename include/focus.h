/*
 * focus.h -- C ABI of the Focus inference hot path for NVIDIA B200 (sm_100a).
 *
 * Focus (arXiv 2604.03260, "Composing Sparse Attention via Learned Grouping") restricts causal
 * attention to pairs that are close (inside a local window) or that share a learned group, and
 * keeps exact softmax over the surviving pairs.  This library is the inference path of one
 * attention layer: group assignment -> tile summaries -> attention forward.
 *
 * General rules for every entry point
 *   - Pointers named "device" must be device memory of the current CUDA device; the caller owns
 *     every buffer.  The library allocates no device memory.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the legacy default
 *     stream).  No entry point synchronises the device.
 *   - Return value: FOCUS_OK (0) or a negative focus_status.  Nothing throws, aborts or traps.
 *     focus_last_error() gives a thread-local message for the last failure.
 *   - Tensors are bf16 with the head dimension D contiguous; the other strides are in elements.
 *     For the attention kernel the base pointer must be 16-byte aligned and every stride a
 *     multiple of 8 elements (TMA requirements).
 *   - Query head h uses KV head h / (Hq / Hkv): consecutive query heads share a KV head.
 *   - Group membership of a token is a uint32 bit mask (bit g = member of group g), K <= 32.
 */
#ifndef FOCUS_H_
#define FOCUS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define FOCUS_API __attribute__((visibility("default")))
#else
#define FOCUS_API
#endif

typedef enum {
    FOCUS_OK = 0,
    FOCUS_ERR_INVALID_ARG = -1, /* null pointer, bad size, Hq % Hkv != 0, topk outside [1,K], misaligned tensor */
    FOCUS_ERR_UNSUPPORTED = -2, /* D not in {64,128,256}, too many mask classes for the sorted layout */
    FOCUS_ERR_CAPACITY = -3,    /* workspace smaller than focus_tiles_workspace_bytes() */
    FOCUS_ERR_ARCH = -4,        /* current device is not compute capability 10.x */
    FOCUS_ERR_CUDA = -5         /* a CUDA call failed; focus_last_error() has its message */
} focus_status;

/* Problem shape.  batch*Hq query heads and batch*Hkv KV heads of n tokens each. */
typedef struct {
    int32_t batch;   /* >= 1 */
    int32_t Hq;      /* query heads, multiple of Hkv */
    int32_t Hkv;     /* key/value heads */
    int32_t n;       /* tokens per sequence, >= 1 */
    int32_t D;       /* head dimension: 64, 128 or 256 */
    int32_t K;       /* number of groups, 1..32 */
    int32_t topk;    /* groups each token joins, 1..K */
    int32_t window;  /* w >= 0: pairs with i - j <= w are always attended (w+1 keys incl. self) */
    float scale;     /* logit scale; 0 selects 1/sqrt(D) */
    float softcap;   /* c > 0: logits become c*tanh(scale*q.k/c) before the softmax; 0 = off */
} focus_shape;

/* A bf16 tensor [batch, H, n, D] in device memory, D contiguous, strides in elements. */
typedef struct {
    void* ptr;
    int64_t stride_b;
    int64_t stride_h;
    int64_t stride_n;
} focus_tensor;

/* Tile sizes of the summaries written by focus_build_tiles (fixed by the ABI). */
#define FOCUS_TILE_M 128
#define FOCUS_TILE_N 128
/* Largest number of distinct mask values per head the class-sorted layout accepts. */
#define FOCUS_MAX_CLASSES 64

#define FOCUS_LAYOUT_ORIGINAL 0
#define FOCUS_LAYOUT_CLASS_SORTED 1
/* Let the library choose from the shape alone (n, K, topk, window): a class-sorted layout when the
 * sequence is long enough for its fixed costs (at least 16384 tokens and 2048 per mask class, 1024 with the separate
 * window pass; C(K, topk) classes assumed) and enough distant pairs fall away (at least half of them for uniform memberships, or at least 15 % from
 * 65536 tokens on); the original layout otherwise.  Of the two class-sorted layouts FOCUS_LAYOUT_SORTED_LOCAL is taken
 * when the window of a block of sorted queries, spread over the C(K-topk, topk) classes it shares no group with,
 * would cost over 1.25 times the key tiles of a window pass in token order, fixed costs included (many classes: K = 8).
 * focus_tiles_layout_of reports the choice in `layout`; pass
 * the same value to focus_tiles_workspace_bytes, focus_build_tiles and focus_attn_fwd. */
#define FOCUS_LAYOUT_AUTO 2
/* Class-sorted layout for the pairs that share a group, plus a second pass in the original token order for the
 * pairs that are attended only because they lie inside the window (no shared group); the two partial results
 * cover disjoint sets of pairs and are joined through their logsumexps (paper Appendix D, "Disjoint decomposition"
 * and "Merge").  With many small classes the sorted order scatters the window of a query block over a wide range
 * of every other class; the separate pass reads the window once, in token order. */
#define FOCUS_LAYOUT_SORTED_LOCAL 3
/* Group-major keys: queries are sorted by class as above, but the keys of a KV head are laid out as K lists, list g
 * holding (in token order) every key that is a member of group g -- a key with several groups is listed once per
 * group.  A block of sorted queries walks the lists of its own groups only, and a pair that shares more than one
 * group is attended under the lowest shared group (in the higher list the key is masked out for that row), so every
 * sharing pair is computed exactly once; the pairs attended only because of the window come from the same second pass
 * in token order as with FOCUS_LAYOUT_SORTED_LOCAL.  With top-k > 1 there are K lists of about n*topk/K keys instead
 * of C(K, topk) class segments of about n/C(K, topk): the padding and the cut tiles at segment ends, which dominate
 * when classes are many and small, fall away, at the price of listing (and staging) every key topk times. */
#define FOCUS_LAYOUT_GROUP_MAJOR 4

/*
 * Byte offsets of the arrays inside a tiles workspace (a pure function of shape and layout;
 * computed on the host, no device access).  nqt = ceil(n/128) query tiles, nkt = ceil(n/128) key
 * tiles, nkw = ceil(nkt/32).  Heads are indexed batch-major (b*H + h).
 */
typedef struct {
    int32_t layout, nqt, nkt, nkw;
    size_t total_bytes;
    size_t counters;   /* uint64[8]: [0] far tile pairs, [1] live far tile pairs, [2] full far tile pairs,
                                     [3] sorted layout: key tiles listed in the ranges, summed over query blocks,
                                     [4] sorted layout: non-zero when a head has more than FOCUS_MAX_CLASSES mask values */
    size_t orq, andq;  /* uint32 [B*Hq][nqt]: OR / AND of the member masks of each query tile */
    size_t ork, andk;  /* uint32 [B*Hkv][nkt] */
    size_t gbits;      /* uint32 [B*Hkv][nkt][K][4]: bit j of word j/32 set when key 128*b + j is in group g */
    size_t live;       /* uint32 [B*Hq][nqt][nkw]: bit b set when (a, b) is a far tile pair that may hold a kept pair */
    size_t live_cnt;   /* int32  [B*Hq][nqt]: popcount of the row of `live` */
    size_t kany, kall; /* uint32 [B*Hkv][K][nkw]: bit b set when key tile b holds a member of group g / only members of g */
    /* class-sorted layouts only (0 otherwise) */
    int32_t nqp, nkp;  /* capacity of the sorted arrays in rows (multiples of 256): n + room for padding every class segment;
                          group-major keys: n*topk + room for padding every list */
    size_t ncls_q, ncls_k;   /* int32 [B*Hq], [B*Hkv]: distinct mask values of the head */
    size_t cls_q, cls_k;     /* uint32 [heads][FOCUS_MAX_CLASSES]: the mask values, ascending */
    size_t cnt_q, cnt_k;     /* int32 [heads][FOCUS_MAX_CLASSES]: tokens of each class */
    /* (group-major keys: "class" j of the key side is group j -- ncls_k = K, cls_k[j] = 1 << j, cnt_k / seg_k / perm_k
       describe the K lists) */
    size_t seg_q, seg_k;     /* int32 [heads][FOCUS_MAX_CLASSES+1]: first sorted slot of each class segment; query
                                segments are padded to multiples of 256 slots, key segments to multiples of 128;
                                entry [ncls] is the number of slots in use */
    size_t perm_q, perm_k;   /* int32 [heads][nqp|nkp]: original position of each sorted slot, ascending inside a
                                segment (stable sort); padding is -1 on the query side and INT32_MAX on the key side */
    size_t qrange;           /* int32 [B*Hq][nqp/256][FOCUS_MAX_CLASSES][2]: first and one-past-last sorted key tile
                                (128 slots) of each key class that a block of 256 sorted queries must visit */
    size_t order;            /* int32 [B*Hkv][(Hq/Hkv)*(nqp/256)][2]: (query head, query block) pairs of each KV head
                                group, most key tiles first */
    size_t gbits_s;          /* FOCUS_LAYOUT_GROUP_MAJOR only: uint32 [B*Hkv][nkp/128][K][4], bit j of word j/32 set when
                                entry 128*b + j of the key lists is a member of group g (like gbits, in list order) */
    size_t qs, ks, vs;       /* bf16 sorted copies [B*Hq][nqp][D], [B*Hkv][nkp][D] x2, filled by focus_attn_fwd */
    size_t scratch;          /* build-time scratch (hash sets of mask values, chunk histograms, block costs) */
    /* FOCUS_LAYOUT_SORTED_LOCAL and FOCUS_LAYOUT_GROUP_MAJOR only (0 otherwise): the two partial results, kept in fp32
       until they are joined */
    size_t o_sorted;         /* fp32 [B*Hq][n][D]: class-sorted pass (its logsumexp goes to the caller's lse) */
    size_t o_local;          /* fp32 [B*Hq][n][D]: window pass */
    size_t lse_local;        /* fp32 [B*Hq][n] */
} focus_tiles_layout;

/* Library version (major*10000 + minor*100 + patch). */
FOCUS_API int focus_version(void);
FOCUS_API const char* focus_status_string(int status);
FOCUS_API const char* focus_last_error(void);

/*
 * focus_assign -- group assignment (paper Sec. 2 "Learned grouping", Eq. 1, with the top-k
 * membership rule of Sec. 2 "Efficiency at inference" / Sec. 3.6).
 * For each head vector x (a query head vector or a key head vector) the score against group g
 * is the cosine between x and centroid g of the vector's KV head; the token joins its `topk` best
 * groups (ties go to the lower group index; a zero vector scores 0 everywhere).
 *   x           device, bf16 [batch, H, n, D]
 *   H           number of heads of x: shape->Hq or shape->Hkv (head h reads centroid set h / (H/Hkv))
 *   centroids   device, fp32 [Hkv, K, D] contiguous; need not be unit length
 *   masks_out   device, uint32 [batch*H, n]
 *   near_ties   device, nullable: *near_ties is incremented (not reset) by the number of vectors whose
 *               margin cos(topk-th) - cos((topk+1)-th), computed in fp32, is below near_tie_eps.
 *               Bit 63 of the word is the kernel's fault flag: it is set when a bounded wait inside the
 *               kernel ran out (4 s) or the kernel found its shared memory misplaced; the masks of the
 *               blocks concerned are then not written.  A caller that passes NULL gets no such report.
 * Arithmetic: the dot products run on the tensor cores with each fp32 centroid split into three bf16
 * terms, so every product with a bf16 vector element is exact and the sums are fp32; |x|, |c_g| and the
 * selection are plain fp32.  Scores agree with the exactly rounded cosine to about 1e-6.
 */
FOCUS_API int focus_assign(const focus_shape* shape, focus_tensor x, int32_t H, const float* centroids,
                 uint32_t* masks_out, unsigned long long* near_ties, float near_tie_eps, void* stream);

/*
 * focus_assign_hidden -- the router in the paper's own form (Sec. 2 "Learned grouping", Eq. 1): one routing
 * vector per token, W_g h_i in d_g dimensions, scored against the centroids C [K, d_g] by dot product; the
 * token joins its `topk` best groups (Sec. 2 "Efficiency at inference"), ties to the lower group index, and
 * every head of the layer, in the query role and in the key role, uses that one mask.  The temperature and the
 * row softmax of Eq. 1 do not change a row's ranking and are not applied.  `bias` (nullable) is added to the
 * scores: Sinkhorn's balanced assignment is diag(r) exp(S/tau) diag(c), whose row ranking is that of
 * S + tau log c, so bias_g = tau log c_g carries the balancing into inference.
 *   shape       batch, Hq, Hkv, n, K, topk are read (D is not used here)
 *   h           device, bf16 hidden states [batch, n, d_model], last dimension contiguous; 16-byte aligned,
 *               strides (elements) multiples of 8; d_model a multiple of 8
 *   Wg          device, fp32 [d_model, d_g] row-major      C   device, fp32 [K, d_g]      bias  device fp32 [K] or NULL
 *   folded      device scratch, fp32 [K, d_model] (K*d_model*4 bytes, 16-byte aligned): receives W_g C_g, the K
 *               vectors the hidden states are scored against (each hidden state is then read once)
 *   mq_out      device uint32 [batch*Hq, n] or NULL     mk_out   device uint32 [batch*Hkv, n] or NULL
 *   near_ties   device, nullable: incremented by the number of tokens whose margin score(topk-th) - score((topk+1)-th),
 *               in fp32 and in score units, is below near_tie_eps; bit 63 is the kernel's fault flag as in focus_assign
 * Arithmetic: as in focus_assign, the dot products run on the tensor cores with each fp32 folded value split into
 * three bf16 terms (exact products, fp32 sums over d_model).
 */
FOCUS_API int focus_assign_hidden(const focus_shape* shape, const void* h, int64_t stride_b, int64_t stride_n,
                                  int32_t d_model, int32_t d_g, const float* Wg, const float* C, const float* bias,
                                  float* folded, uint32_t* mq_out, uint32_t* mk_out, unsigned long long* near_ties,
                                  float near_tie_eps, void* stream);

/*
 * focus_tiles_layout_of -- host-only: sizes and offsets of the tiles workspace.
 * focus_tiles_workspace_bytes -- its total_bytes (0 on bad arguments).
 */
FOCUS_API int focus_tiles_layout_of(const focus_shape* shape, int32_t layout, focus_tiles_layout* out);
FOCUS_API size_t focus_tiles_workspace_bytes(const focus_shape* shape, int32_t layout);

/*
 * focus_build_tiles -- per-tile summaries of the membership masks and the live far-tile set
 * (paper Sec. 2 "Efficiency at inference": different-group distant pairs are never computed;
 * Sec. 2 item "Group": stable sort of tokens by group for the class-sorted layout).
 * A tile pair (a, b) is "far" when every pair in it has i - j > w.  A far pair is live iff
 * OR(query tile masks) & OR(key tile masks) != 0; dead far pairs hold no attended pair.
 *   mq   device, uint32 [batch*Hq, n]    mk   device, uint32 [batch*Hkv, n]
 *   layout  FOCUS_LAYOUT_ORIGINAL, or FOCUS_LAYOUT_CLASS_SORTED (tokens stably sorted by mask value
 *           per head, so that a tile holds one mask class and tile pairs are all-share or none-share),
 *           or FOCUS_LAYOUT_SORTED_LOCAL (the same arrays, with only the sharing classes listed in `qrange`),
 *           or FOCUS_LAYOUT_AUTO
 *   ws   device workspace of ws_bytes >= focus_tiles_workspace_bytes(shape, layout), 256-byte aligned.
 *        Contents are described by focus_tiles_layout.  The workspace is tied to (shape, mq, mk).
 */
FOCUS_API int focus_build_tiles(const focus_shape* shape, const uint32_t* mq, const uint32_t* mk, int32_t layout,
                      void* ws, size_t ws_bytes, void* stream);

/*
 * focus_attn_fwd -- causal attention forward over the attended pairs (paper Sec. 2 and
 * Appendix D, first equation): pair (i, j) is attended iff
 *        j <= i  and  ( i - j <= window  or  mq[h,i] & mk[kv(h),j] != 0 ).
 * s_ij = scale*q_i.k_j (then softcap*tanh(s_ij/softcap) if softcap > 0);
 * lse_i = log sum_j exp(s_ij); o_i = sum_j exp(s_ij - lse_i) v_j over attended j: exact softmax,
 * no renormalisation.  bf16 operands, fp32 accumulation, probabilities rounded to bf16 before PV.
 *   q, o        device bf16 [batch, Hq, n, D]      k, v   device bf16 [batch, Hkv, n, D]
 *   mq, mk      device masks; may be NULL when tiles_ws is NULL
 *   tiles_ws    workspace written by focus_build_tiles for the same shape and masks.  NULL = dense
 *               causal mode (every causal pair attended; masks and layout ignored).
 *   layout      the layout the workspace was built with (FOCUS_LAYOUT_SORTED_LOCAL: the class-sorted pass over
 *               sharing pairs, the window pass in token order, then a merge kernel): FOCUS_LAYOUT_ORIGINAL walks tiles in token
 *               order and skips dead far tiles; FOCUS_LAYOUT_CLASS_SORTED gathers Q/K/V into the
 *               class-sorted order kept in the workspace, walks only sharing class pairs plus the
 *               window, and scatters O/lse back to token order.
 *   lse         device fp32 [batch*Hq, n], natural log
 *   dev_status  device int32[4], nullable: [0] stays 0 on success.  [0] = 1: a bounded wait inside the
 *               kernel expired (the kernel then drains and exits; outputs are invalid), [1] = code of
 *               the wait (10, 11: the load role waiting for a free query buffer / ring slot; 20-26: the
 *               MMA role waiting for queries, a ring stage or probabilities; 30-41: a softmax role
 *               waiting for S, its partner thread or O), [2] = work item, [3] = CTA.  [0] = 2: a class-sorted layout was asked for
 *               but a head holds more than FOCUS_MAX_CLASSES distinct mask values (possible only with
 *               masks that do not come from a top-k rule); nothing was computed and O / lse were not
 *               written.  dev_status must not be NULL with a tiles workspace in any layout but
 *               FOCUS_LAYOUT_ORIGINAL (FOCUS_ERR_INVALID_ARG otherwise).  The caller zeroes it and reads
 *               it after synchronising.
 */
FOCUS_API int focus_attn_fwd(const focus_shape* shape, focus_tensor q, focus_tensor k, focus_tensor v,
                   const uint32_t* mq, const uint32_t* mk, const void* tiles_ws, int32_t layout,
                   focus_tensor o, float* lse, int32_t* dev_status, void* stream);

/*
 * focus_decode_step -- one generation step: the newest token (position n-1, its key and value already appended
 * to the caches) as the only query, under the same rule as focus_attn_fwd (paper Sec. 2 "Efficiency at inference",
 * Appendix D first equation): key j is attended iff n-1-j <= window or mq_new[h] & mk[kv(h), j] != 0; exact softmax
 * over the attended keys; bf16 operands, fp32 accumulation, probabilities rounded to bf16 before P V.  The paper evaluates generation with the method but
 * gives no procedure; this is the forward rule applied to one row.  Only attended K/V rows are read from HBM.
 *   shape       n = cached tokens including the new one; Hq / Hkv <= 8
 *   q, o        device bf16 [batch, Hq, D]: ptr, stride_b, stride_h are used (stride_n ignored)
 *   k, v        device bf16 caches [batch, Hkv, n, D]; rows 16-byte aligned (ptr 16-byte aligned, strides multiples of 8)
 *   mq_new      device uint32 [batch*Hq]: membership mask of the new token per query head
 *   mk          device uint32 [batch*Hkv, n]: membership masks of the cached keys
 *   lse         device fp32 [batch*Hq], natural log
 *   ws          device scratch of at least focus_decode_workspace_bytes(shape) bytes, 16-byte aligned (partial results
 *               of the key splits); contents need not be preserved between calls
 */
FOCUS_API size_t focus_decode_workspace_bytes(const focus_shape* shape);
FOCUS_API int focus_decode_step(const focus_shape* shape, focus_tensor q, focus_tensor k, focus_tensor v,
                                const uint32_t* mq_new, const uint32_t* mk, focus_tensor o, float* lse, void* ws,
                                size_t ws_bytes, void* stream);

/*
 * focus_count_kept -- exact number of attended pairs per query head (the denominator-free
 * numerator of "effective FLOP": 4*D flop per attended pair).  Uses the gbits summaries of a
 * workspace built for the same shape and masks (either layout).
 *   counts_out  device uint64 [batch*Hq]; overwritten.
 */
FOCUS_API int focus_count_kept(const focus_shape* shape, const uint32_t* mq, const void* tiles_ws,
                     unsigned long long* counts_out, void* stream);

/*
 * focus_count_kept_noalloc -- the paper has no counterpart; this is a convenience of the library.
 * Same result as focus_count_kept, for callers that cannot allocate device memory: code that was
 * handed its input and output buffers by a host framework and owns no allocator, a server whose
 * device arena is fully committed at start-up, or a latency-critical loop in which cudaMalloc is
 * off limits because it synchronises the device.  Instead of reading the group bitmaps from a
 * caller-allocated tiles workspace, this entry point builds them from mk into a fixed array that is
 * part of the library image (FOCUS_NOALLOC_MAX_BYTES, resident on every device that loads the
 * library until the process exits).  It calls no allocating routine.
 *   mq          device, uint32 [batch*Hq, n]       mk   device, uint32 [batch*Hkv, n]
 *   counts_out  device uint64 [batch*Hq]; overwritten
 * Limit: batch*Hkv*ceil(n/128)*K*16 bytes must fit in FOCUS_NOALLOC_MAX_BYTES, otherwise
 * FOCUS_ERR_CAPACITY is returned and nothing is launched (1 MiB covers the 128K-token metric point:
 * 8 KV heads x 1024 tiles x 4 groups x 16 B = 512 KiB).
 * batch*Hq and batch*Hkv must not exceed 65535 (FOCUS_ERR_UNSUPPORTED otherwise, nothing launched).
 * The first call on each device looks up the array's device address (with that device current)
 * and keeps it for the life of the process; make that first call outside any stream capture, and
 * do not call this entry point again on a device whose context the application has destroyed
 * (cudaDeviceReset): the remembered address is then stale.  All calls share the one array, which keeps the
 * previous call's contents; each call rewrites the part it reads, so stale contents are harmless,
 * but two calls whose kernels may overlap on the GPU (different streams) race on it.
 */
#define FOCUS_NOALLOC_MAX_BYTES (1 << 20)
FOCUS_API int focus_count_kept_noalloc(const focus_shape* shape, const uint32_t* mq, const uint32_t* mk,
                                       unsigned long long* counts_out, void* stream);

/*
 * Training-time forward (paper Sec. 2 "Learned grouping" and "Gated attention", Eq. 1 and Eq. 2).  During
 * training nothing is pruned: every causal pair is computed and the score of a distant pair is multiplied by a
 * gate built from soft group assignments, so this path has no speedup over dense attention (the paper says so).
 *
 * focus_router_scores -- S[b, i, g] = (W_g h_i) . C_g, the argument of Eq. 1's normalisation, in fp32 on the
 * exact bf16 hidden states.  Arguments as for focus_assign_hidden;
 *   scores_out  device fp32 [batch, n, ld], ld = 4 for K <= 4, else 8 for K <= 8, else 16 or 32 (the smallest
 *               that holds K); entries g >= K are written as 0.  16-byte aligned.
 *
 * focus_sinkhorn -- the Sinkhorn normalisation of Sec. 2: Q = exp(S / tau); `iters` times divide every column
 * by its sum over the tokens of the sequence, then every row by its sum over the groups.  Each sequence of the
 * batch is normalised on its own.  Computed in the log domain (offsets per token and per group, fp32, column
 * sums accumulated in fp64), which is the same arithmetic without overflow; after the first row division every
 * entry lies in (0, 1].
 *   shape       batch, n, K are read             scores   device fp32 [batch, n, ld] (ld as above)
 *   tau > 0, iters >= 1 (the paper uses tau = 0.1, iters = 10)
 *   ws          device scratch, focus_sinkhorn_workspace_bytes(shape, iters) bytes, 16-byte aligned
 *   g_out       device fp32 [batch, n, ld]; entries g >= K are written as 0; may be the scores buffer itself
 *
 * focus_gate_attn_fwd -- Eq. 2: for j <= i
 *        s_ij = scale * q_i.k_j * ( 1 if i - j <= window, else sigmoid(lambda * g_i.g_j) ),
 * then exact row softmax over all j <= i, o_i = sum_j p_ij v_j, lse_i = log sum_j exp(s_ij).  The equation is
 * followed as printed: two orthogonal assignments give the gate sigmoid(0) = 1/2.  Same kernel, operand
 * precision and accumulation as focus_attn_fwd in dense causal mode; the gate is evaluated in fp32 as
 * 1/2 + 1/2 tanh(lambda/2 g_i.g_j) with the hardware tanh approximation.
 *   shape       softcap must be 0; K <= 32, and K <= 16 at D = 256 (FOCUS_ERR_UNSUPPORTED otherwise); masks and topk
 *               are not used
 *   q, k, v, o, lse, dev_status   as for focus_attn_fwd
 *   g           device fp32 [batch, n, ld], ld = focus_soft_ld(K) (4, 8, 16 or 32); one assignment per token, shared by all heads;
 *               entries g >= K must be 0 (focus_sinkhorn writes them so); 16-byte aligned
 */
FOCUS_API int focus_router_scores(const focus_shape* shape, const void* h, int64_t stride_b, int64_t stride_n,
                                  int32_t d_model, int32_t d_g, const float* Wg, const float* C, float* folded,
                                  float* scores_out, void* stream);
FOCUS_API int32_t focus_soft_ld(int32_t K);     /* the row length ld for K groups (4, 8, 16 or 32; 0 if K is out of range) */
FOCUS_API size_t focus_sinkhorn_workspace_bytes(const focus_shape* shape, int32_t iters);
FOCUS_API int focus_sinkhorn(const focus_shape* shape, const float* scores, float tau, int32_t iters, void* ws,
                             size_t ws_bytes, float* g_out, void* stream);
FOCUS_API int focus_gate_attn_fwd(const focus_shape* shape, focus_tensor q, focus_tensor k, focus_tensor v,
                                  const float* g, float lambda, focus_tensor o, float* lse, int32_t* dev_status,
                                  void* stream);

/*
 * focus_sinkhorn_bwd -- the derivative of focus_sinkhorn (paper Sec. 2 "Learned grouping": the soft assignments are
 * trained through the Sinkhorn steps).  Given dg = d loss / d g for g = sinkhorn(scores, tau, iters), writes
 * d loss / d scores.  Each step "divide by the sum along an axis", Z = X / sum(X), is differentiated as
 * dX = (dZ - sum(dZ * Z)) / sum(X) along that axis, the `iters` column and row divisions in reverse order, and the
 * exponential last: dS = dQ0 * exp(S / tau) / tau.  The iterates are not stored: a row of any iterate follows from its
 * score row and the column sums of the forward passes, which this call recomputes into `ws` first (it does not need
 * focus_sinkhorn to have run).  fp32 per row, column sums in fp64; offsets kept as logarithms as in the forward.
 *   scores       device fp32 [batch, n, ld], ld = focus_soft_ld(K), as given to focus_sinkhorn; read only
 *   ws           device scratch, focus_sinkhorn_bwd_workspace_bytes(shape, iters) bytes, 16-byte aligned
 *   dg           device fp32 [batch, n, ld]; entries g >= K are ignored
 *   dscores_out  device fp32 [batch, n, ld]; entries g >= K are written as 0; may be the dg buffer, not the scores
 * The derivatives of the gated attention itself (Eq. 2) have an oracle and pins only; no kernel computes them.
 */
FOCUS_API size_t focus_sinkhorn_bwd_workspace_bytes(const focus_shape* shape, int32_t iters);
FOCUS_API int focus_sinkhorn_bwd(const focus_shape* shape, const float* scores, float tau, int32_t iters, void* ws,
                                 size_t ws_bytes, const float* dg, float* dscores_out, void* stream);

/*
 * focus_selftest_umma -- diagnostic, not on the hot path (the paper has no counterpart): one
 * 128 x 128 x D tile S = A B^T and one 128 x D x 128 tile O = P V through the same TMA, descriptor
 * and tcgen05 building blocks as focus_attn_fwd, so that an encoding mistake shows up in isolation.
 *   a, b, v   device bf16 [128, D] row-major     p   device bf16 [128, 128] row-major
 *   s_out     device fp32 [128, 128]             o_out   device fp32 [128, D]
 *   dev_status device int32, zeroed by the caller; non-zero if a bounded wait expired
 */
FOCUS_API int focus_selftest_umma(int32_t D, const void* a, const void* b, const void* p, const void* v, float* s_out,
                        float* o_out, int32_t* dev_status, void* stream);

/*
 * focus_selftest_stalled_wait -- diagnostic (the paper has no counterpart): runs the attention kernel in dense causal
 * mode with one stage of its K/V ring deliberately left unfilled, so that the role waiting for that stage runs into
 * its time limit.  Every wait inside the attention kernels is bounded (4 s in focus_attn_fwd); this entry point sets
 * the bound to `wait_limit_ns` and shows the exit taken when it expires: dev_status[0] = 1, [1] = code of the wait
 * that gave up, [2] = work item, [3] = CTA; the other roles of the CTA notice, nothing traps or hangs, tensor memory
 * is released and the kernel returns.  O and lse are left incomplete.  The device and the context stay usable.
 *   shape, q, k, v, o, lse   as for focus_attn_fwd (n >= 512; masks are not used)
 *   wait_limit_ns            1000 ... 4000000000; the bound is checked at a granularity of about 0.1 s
 *   dev_status               device int32[4], zeroed by the caller, required
 */
FOCUS_API int focus_selftest_stalled_wait(const focus_shape* shape, focus_tensor q, focus_tensor k, focus_tensor v,
                                          focus_tensor o, float* lse, unsigned long long wait_limit_ns,
                                          int32_t* dev_status, void* stream);

/*
 * focus_selftest_umma_pair -- diagnostic (the paper has no counterpart): the same two tiles with D = 128 through one
 * MMA shared by a pair of CTAs on neighbouring SMs (a form focus_attn_fwd does not use): 256 rows of A and P (128
 * per CTA), each CTA staging half of B (64 of its 128 rows) and half of V (64 of its 128 columns).
 *   a, p      device bf16 [256, 128] row-major     b, v   device bf16 [128, 128] row-major
 *   s_out, o_out   device fp32 [256, 128]          dev_status   as above
 */
FOCUS_API int focus_selftest_umma_pair(const void* a, const void* b, const void* p, const void* v, float* s_out,
                                       float* o_out, int32_t* dev_status, void* stream);

/*
 * focus_selftest_mma_rate -- diagnostic (the paper has no counterpart): the rate at which the tensor pipe works off
 * tcgen05 MMAs when nothing else runs, in the shapes the attention kernel uses or could use.  One CTA (pair = 0) or CTA
 * pair (pair = 1, M = 256) per SM issues `rounds` rounds of MMA chains on operands resident in shared and tensor
 * memory; a chain is eight K = 16 instructions = one 128 x N x 128 product (256 x N x 128 across a pair).
 *   N         64, 96, 128 or 256 (pairs: 128 or 256)
 *   ts        0: both operands from shared memory, K-major (S = Q K^T); 1: A from tensor memory, B MN-major (O = P V), N <= 128
 *   pattern   0: one chain per commit, two commits in flight; 1: two chains of the first form per commit, instructions
 *             alternating; 2: one chain of each form per commit, alternating; 3: one of each, one after the other
 *             (patterns 1-3: four chains in flight, ts = 0, N <= 128)
 *   rounds    2 ... 1000000
 *   result    device, three 64-bit words, written by CTA 0: clock cycles, nanoseconds, fault flag (1 if a wait of the
 *             probe ran out after 1 s; the kernel then drains and returns)
 * flop per clock and SM = chains per round x 2 x 128 x N x 128 x rounds / cycles (nominal bf16 rate: 8192).
 */
FOCUS_API int focus_selftest_mma_rate(int32_t pair, int32_t N, int32_t ts, int32_t pattern, int32_t rounds,
                                      unsigned long long* result, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* FOCUS_H_ */
