"""Focus oracle -- TEST INFRASTRUCTURE, not part of the product.

Python face of the fp64 CPU oracle.  The per-row attention and the group assignment are the C
functions in ``focus_oracle.c`` (called through ctypes); the remaining pieces are plain numpy.
Nothing here imports, links or shares code with the CUDA library, and the product never imports
this module: only the tests, the smoke check and the bench's CPU-baseline leg do.

Passages of the paper each function follows:

* ``assign``            Sec. 2 "Learned grouping" (Eq. 1) + the top-k membership rule of Sec. 2
                        "Efficiency at inference" and Sec. 3.6.
* ``assign_hidden``     Sec. 2 "Learned grouping", Eq. 1 as the paper states it: one routing vector per token,
                        ``W_g h_i`` in d_g dimensions, scored against ``C`` by dot product; top-k of the scores
                        (row-softmax and the temperature do not change a row's ranking).  The optional per-group
                        bias is what Sinkhorn's column scaling leaves behind at inference: the balanced
                        assignment is diag(r) exp(S/tau) diag(c), whose row ranking is that of S + tau log c.
* ``attn_rows``         Sec. 2 (exact softmax over attended pairs) + Appendix D, first equation
                        (the hard Focus mask), with "same group" read as "membership sets intersect".
* ``dense_brute``       the O(n^2) masked reference the paper verifies against (Appendix D,
                        "Empirical verification"): explicit n x n boolean matrix, textbook softmax.
* ``ab_merge``          Appendix D "Disjoint decomposition" and "Merge": sets A (same-group causal)
                        and B (cross-group local) computed separately and joined through their
                        logsumexps.  Defined by the paper for single-group assignment only.
* ``kept_pairs``        size of the attended set of Appendix D's mask (exact integer count).
* ``tile_reference``    the per-tile mask summaries and the far-tile liveness rule (a far tile can be
                        dropped when no query of the tile shares a group with any key of the tile);
                        this is the tile-level consequence of Sec. 2 "different-group distant pairs
                        are never computed".
* ``class_sort``        Sec. 2 "Sort tokens by group (stable sort preserves causal order)".
* ``sorted_layout``     the padded class-sorted arrays and, per block of sorted queries and key class, the
                        range of sorted key tiles that can hold an attended pair -- the same Sec. 2 sort
                        combined with Appendix D's mask (same-class-sharing keys up to the block's last
                        position; other keys only inside the window).

* ``group_major_layout`` the same Sec. 2 sort with a token that belongs to several groups (top-k > 1, Sec. 3.6)
                        listed once per group: K key lists in token order; a block of sorted queries reads the lists
                        of its own groups up to its last position, and a pair sharing several groups is attended under
                        the lowest shared one.  Covers exactly the sharing pairs of Appendix D's mask, each once.

* ``router_scores``     Sec. 2 "Learned grouping", the argument of Eq. 1's normalisation: (W_g h_i) . C_g.
* ``sinkhorn``          Sec. 2 "Learned grouping", the two-step Sinkhorn normalisation: exponentiate the scores
                        over the temperature, then N times divide by the sums over tokens and by the sums over
                        groups, in that order.
* ``gated_attn``        Sec. 2 "Gated attention" (Eq. 2), the training-time forward over all causal pairs: the
                        score of a distant pair is multiplied by sigmoid(lambda g_i . g_j), a pair inside the
                        window keeps its score.  The equation is followed as printed, so the gate of two
                        orthogonal assignments is sigmoid(0) = 1/2 (the prose around it speaks of zero).

* ``sinkhorn_backward`` / ``gated_attn_backward``
                        the derivatives of the two functions above (chain rule through every division of the
                        Sinkhorn steps; through the row softmax, the gate sigmoid(lambda g_i . g_j) and the score of
                        Eq. 2).  No kernel computes them yet: they are the reference a backward pass would be
                        checked against, pinned by finite differences and by automatic differentiation.

Parity status: every function above is pinned by the CPU tests.  "parity unpinned": the paper's
perplexity and benchmark numbers (datasets and trained weights are not available).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "focus_oracle.c")
_LIB = os.path.join(_HERE, "libfocus_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile focus_oracle.c with gcc into libfocus_oracle.so beside it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        c_i64, c_int, c_dbl, vp = ctypes.c_int64, ctypes.c_int, ctypes.c_double, ctypes.c_void_p
        lib.focus_oracle_threads.restype = c_int
        lib.focus_oracle_assign.restype = c_int
        lib.focus_oracle_assign.argtypes = [vp, c_int, c_int, c_i64, c_int, vp, c_int, c_int, vp, vp]
        lib.focus_oracle_attn_rows.restype = c_int
        lib.focus_oracle_attn_rows.argtypes = [vp, vp, vp, c_int, c_int, c_i64, c_int, vp, vp, c_i64,
                                               c_dbl, c_dbl, c_i64, vp, vp, vp, vp, vp, vp]
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().focus_oracle_threads())


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64, exactly."""
    u = bits.astype(np.uint32) << 16
    return u.view(np.float32).astype(np.float64)


def assign(x_bits: np.ndarray, centroids: np.ndarray, topk: int):
    """x_bits uint16 [H, n, D], centroids float32 [Hkv, K, D] -> (masks uint32 [H, n], margins f64 [H, n])."""
    x_bits = _c(x_bits, np.uint16)
    centroids = _c(centroids, np.float32)
    H, n, D = x_bits.shape
    Hkv, K, D2 = centroids.shape
    assert D2 == D
    masks = np.zeros((H, n), np.uint32)
    margins = np.zeros((H, n), np.float64)
    rc = _load().focus_oracle_assign(_ptr(x_bits), H, Hkv, n, D, _ptr(centroids), K, topk,
                                     _ptr(masks), _ptr(margins))
    if rc != 0:
        raise ValueError("focus_oracle_assign: bad arguments")
    return masks, margins


def attn_rows(q_bits, k_bits, v_bits, mq, mk, window, scale=None, softcap=0.0, rows=None):
    """Attention rows from the definition.

    q_bits uint16 [Hq, n, D]; k_bits, v_bits uint16 [Hkv, n, D]; mq uint32 [Hq, n]; mk uint32 [Hkv, n].
    rows: int array [R, 2] of (head, token) pairs, or None for every row (head-major order).
    Returns dict(O f64 [R, D], lse f64 [R], psum f64 [R], kept int64 [R], rows [R, 2]).
    """
    q_bits = _c(q_bits, np.uint16); k_bits = _c(k_bits, np.uint16); v_bits = _c(v_bits, np.uint16)
    mq = _c(mq, np.uint32); mk = _c(mk, np.uint32)
    Hq, n, D = q_bits.shape
    Hkv = k_bits.shape[0]
    assert k_bits.shape == (Hkv, n, D) and v_bits.shape == (Hkv, n, D)
    assert mq.shape == (Hq, n) and mk.shape == (Hkv, n)
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    if rows is None:
        hh, ii = np.meshgrid(np.arange(Hq), np.arange(n), indexing="ij")
        rows = np.stack([hh.ravel(), ii.ravel()], axis=1)
    rows = np.asarray(rows, dtype=np.int64).reshape(-1, 2)
    R = rows.shape[0]
    row_h = _c(rows[:, 0], np.int32); row_i = _c(rows[:, 1], np.int64)
    O = np.zeros((R, D), np.float64); lse = np.zeros(R, np.float64)
    psum = np.zeros(R, np.float64); kept = np.zeros(R, np.int64)
    rc = _load().focus_oracle_attn_rows(_ptr(q_bits), _ptr(k_bits), _ptr(v_bits), Hq, Hkv, n, D,
                                        _ptr(mq), _ptr(mk), int(window), float(scale), float(softcap),
                                        R, _ptr(row_h), _ptr(row_i), _ptr(O), _ptr(lse), _ptr(psum),
                                        _ptr(kept))
    if rc != 0:
        raise ValueError("focus_oracle_attn_rows: bad arguments")
    return dict(O=O, lse=lse, psum=psum, kept=kept, rows=rows)


# ----------------------------------------------------------------------------------------------
# numpy pieces
# ----------------------------------------------------------------------------------------------

def kept_matrix(mq_h: np.ndarray, mk_h: np.ndarray, window: int) -> np.ndarray:
    """Explicit n x n boolean mask of Appendix D's first equation for one (q head, kv head) pair."""
    n = mq_h.shape[0]
    i = np.arange(n)[:, None]
    j = np.arange(n)[None, :]
    share = (mq_h[:, None] & mk_h[None, :]) != 0
    return (j <= i) & (((i - j) <= window) | share)


def dense_brute(q_bits, k_bits, v_bits, mq, mk, window, scale=None, softcap=0.0):
    """O(n^2) masked reference: explicit mask, -inf elsewhere, full-row textbook softmax, times V.

    Returns (O f64 [Hq, n, D], lse f64 [Hq, n]).  Small n only.
    """
    Hq, n, D = q_bits.shape
    Hkv = k_bits.shape[0]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    Q = bf16_bits_to_f64(np.asarray(q_bits)); Kd = bf16_bits_to_f64(np.asarray(k_bits))
    V = bf16_bits_to_f64(np.asarray(v_bits))
    O = np.zeros((Hq, n, D)); L = np.zeros((Hq, n))
    for h in range(Hq):
        hk = h // G
        S = scale * (Q[h] @ Kd[hk].T)
        if softcap > 0:
            S = softcap * np.tanh(S / softcap)
        M = kept_matrix(np.asarray(mq)[h], np.asarray(mk)[hk], window)
        S = np.where(M, S, -np.inf)
        mx = S.max(axis=1, keepdims=True)
        E = np.exp(S - mx)
        Z = E.sum(axis=1, keepdims=True)
        O[h] = (E / Z) @ V[hk]
        L[h] = (mx + np.log(Z))[:, 0]
    return O, L


def ab_merge(q_bits, k_bits, v_bits, g, window, scale=None, double_count=False):
    """Appendix D two-set path for single-group assignment g [n] (one head, MHA).

    Set A = same-group causal pairs, set B = cross-group pairs inside the window; each set gets its
    own softmax attention and logsumexp, joined by the Appendix D merge formula.  With
    ``double_count=True`` set B is replaced by *all* local pairs (the overlapping decomposition the
    paper rejects), which counts same-group local pairs twice.
    q_bits/k_bits/v_bits uint16 [n, D].  Returns (O [n, D], lse [n]).
    """
    n, D = q_bits.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    Q = bf16_bits_to_f64(q_bits); Kd = bf16_bits_to_f64(k_bits); V = bf16_bits_to_f64(v_bits)
    S = scale * (Q @ Kd.T)
    i = np.arange(n)[:, None]; j = np.arange(n)[None, :]
    causal = j <= i
    same = g[:, None] == g[None, :]
    local = (i - j) <= window
    A = causal & same
    B = causal & local & (np.ones_like(same) if double_count else ~same)

    def part(M):
        Sm = np.where(M, S, -np.inf)
        mx = Sm.max(axis=1, keepdims=True)
        has = np.isfinite(mx)
        mx0 = np.where(has, mx, 0.0)
        E = np.where(M, np.exp(Sm - mx0), 0.0)
        Z = E.sum(axis=1, keepdims=True)
        o = np.where(has, (E @ V) / np.where(Z > 0, Z, 1.0), 0.0)
        l = np.where(has[:, 0], mx0[:, 0] + np.log(np.where(Z[:, 0] > 0, Z[:, 0], 1.0)), -np.inf)
        return o, l

    oA, lA = part(A)
    oB, lB = part(B)
    mx = np.maximum(lA, lB)
    eA = np.exp(lA - mx); eB = np.exp(lB - mx)
    O = (eA[:, None] * oA + eB[:, None] * oB) / (eA + eB)[:, None]
    return O, mx + np.log(eA + eB)


def kept_pairs(mq: np.ndarray, mk: np.ndarray, window: int) -> np.ndarray:
    """Exact number of attended pairs per query head (int64 [Hq]).

    Row i keeps its min(i, w) + 1 local keys plus every key j < i - w whose membership mask meets
    the row's; the second term is read from a running count of far keys per distinct key mask.
    """
    mq = np.asarray(mq, np.uint32); mk = np.asarray(mk, np.uint32)
    Hq, n = mq.shape
    Hkv = mk.shape[0]
    G = Hq // Hkv
    out = np.zeros(Hq, np.int64)
    idx = np.arange(n, dtype=np.int64)
    far_len = np.maximum(idx - window, 0)            # number of keys j with i - j > w
    local = np.minimum(idx, window) + 1
    for h in range(Hq):
        hk = h // G
        total = int(local.sum())
        kvals = np.unique(mk[hk])
        for qv in np.unique(mq[h]):
            sharing = kvals[(kvals & qv) != 0]
            if sharing.size == 0:
                continue
            is_share = np.isin(mk[hk], sharing)
            cum = np.concatenate([[0], np.cumsum(is_share, dtype=np.int64)])   # cum[m] = # sharing keys j < m
            rows = mq[h] == qv
            total += int(cum[far_len[rows]].sum())
        out[h] = total
    return out


def tile_reference(mq: np.ndarray, mk: np.ndarray, window: int, BM: int, BN: int):
    """Tile summaries and far-tile liveness, straight from their definitions.

    Query tile a covers rows [a*BM, min(n, (a+1)*BM)), key tile b covers keys [b*BN, min(n, (b+1)*BN)).
    Returns dict with
      orq, andq  uint32 [Hq, nqt]   OR / AND of the member masks of each query tile
      ork, andk  uint32 [Hkv, nkt]
      far        bool [nqt, nkt]    every pair of the tile pair has i - j > w (so it is causal too)
      live       bool [Hq, nqt, nkt] far and (orq & ork != 0)
      full       bool [Hq, nqt, nkt] far and (andq & andk != 0): every pair shares a group
    """
    mq = np.asarray(mq, np.uint32); mk = np.asarray(mk, np.uint32)
    Hq, n = mq.shape
    Hkv = mk.shape[0]
    G = Hq // Hkv
    nqt = (n + BM - 1) // BM
    nkt = (n + BN - 1) // BN

    def summarise(m, T, nt):
        o = np.zeros((m.shape[0], nt), np.uint32); a = np.zeros((m.shape[0], nt), np.uint32)
        for t in range(nt):
            seg = m[:, t * T:min(n, (t + 1) * T)]
            o[:, t] = np.bitwise_or.reduce(seg, axis=1)
            a[:, t] = np.bitwise_and.reduce(seg, axis=1)
        return o, a

    orq, andq = summarise(mq, BM, nqt)
    ork, andk = summarise(mk, BN, nkt)
    qmin = np.arange(nqt) * BM
    kmax = np.minimum(n, (np.arange(nkt) + 1) * BN) - 1
    far = (qmin[:, None] - kmax[None, :]) > window
    live = np.zeros((Hq, nqt, nkt), bool); full = np.zeros((Hq, nqt, nkt), bool)
    for h in range(Hq):
        hk = h // G
        live[h] = far & ((orq[h][:, None] & ork[hk][None, :]) != 0)
        full[h] = far & ((andq[h][:, None] & andk[hk][None, :]) != 0)
    return dict(orq=orq, andq=andq, ork=ork, andk=andk, far=far, live=live, full=full)


def class_sort(m_h: np.ndarray):
    """Stable sort of one head's tokens by membership-mask value.

    Returns (perm int64 [n], classes uint32 [C], counts int64 [C]): perm lists original positions,
    class by class (classes ascending by mask value), positions ascending inside a class.
    """
    m_h = np.asarray(m_h, np.uint32)
    perm = np.argsort(m_h, kind="stable").astype(np.int64)
    classes, counts = np.unique(m_h, return_counts=True)
    return perm, classes.astype(np.uint32), counts.astype(np.int64)


def sorted_layout(mq_h: np.ndarray, mk_h: np.ndarray, window: int, pad_q: int = 256, pad_k: int = 128,
                  tile: int = 128):
    """Class-sorted layout of one (query head, KV head) pair, written from its definition.

    Tokens are stably sorted by mask value; each class segment is padded to a multiple of ``pad_q``
    (queries, padding -1) or ``pad_k`` (keys, padding INT32_MAX).  For every block of ``pad_q`` sorted
    queries (one class, positions pmin..pmax) and every key class: if the two mask values intersect,
    the keys of the class with position <= pmax can be attended; otherwise only those with position
    in [pmin - window, pmax].  The range is given in sorted key tiles of ``tile`` slots,
    (first, one past last), (0, 0) when empty.
    Returns dict(cls_q, cnt_q, seg_q, perm_q, cls_k, cnt_k, seg_k, perm_k, ranges [nblk, ncls_k, 2]).
    """
    def side(m, pad, fill):
        perm, cls, cnt = class_sort(m)
        seg = np.zeros(len(cls) + 1, np.int64)
        seg[1:] = np.cumsum((cnt + pad - 1) // pad * pad)
        out = np.full(int(seg[-1]), fill, np.int64)
        src = 0
        for c in range(len(cls)):
            out[seg[c]:seg[c] + cnt[c]] = perm[src:src + cnt[c]]
            src += cnt[c]
        return cls, cnt, seg, out

    cls_q, cnt_q, seg_q, perm_q = side(np.asarray(mq_h, np.uint32), pad_q, -1)
    cls_k, cnt_k, seg_k, perm_k = side(np.asarray(mk_h, np.uint32), pad_k, np.iinfo(np.int32).max)
    nblk = int(seg_q[-1]) // pad_q
    ranges = np.zeros((nblk, len(cls_k), 2), np.int64)
    for blk in range(nblk):
        rows = perm_q[blk * pad_q:(blk + 1) * pad_q]
        rows = rows[rows >= 0]
        jq = int(np.searchsorted(seg_q, blk * pad_q, side="right")) - 1
        pmin, pmax = int(rows.min()), int(rows.max())
        for jk in range(len(cls_k)):
            kp = perm_k[seg_k[jk]:seg_k[jk] + cnt_k[jk]]
            if int(cls_q[jq]) & int(cls_k[jk]):
                idx = np.nonzero(kp <= pmax)[0]
            else:
                idx = np.nonzero((kp <= pmax) & (kp >= pmin - window))[0]
            if idx.size:
                ranges[blk, jk] = ((seg_k[jk] + idx.min()) // tile, (seg_k[jk] + idx.max()) // tile + 1)
    return dict(cls_q=cls_q, cnt_q=cnt_q, seg_q=seg_q, perm_q=perm_q, cls_k=cls_k, cnt_k=cnt_k, seg_k=seg_k,
                perm_k=perm_k, ranges=ranges)


def group_major_layout(mq_h: np.ndarray, mk_h: np.ndarray, K: int, pad_q: int = 256, pad_k: int = 128, tile: int = 128):
    """Group-major key lists of one (query head, KV head) pair, written from their definition.

    Queries: stably sorted by mask value, class segments padded to ``pad_q`` (padding -1), as in ``sorted_layout``.
    Keys: list g (g = 0..K-1) holds the positions of the keys that are members of group g, ascending, padded to a
    multiple of ``pad_k`` with INT32_MAX; the lists follow one another.  ``gbits`` [tiles, K, tile] says for every
    list entry which groups its key belongs to.  ``ranges`` [nblk, K, 2]: for a block of ``pad_q`` sorted queries of
    class c and every group g in c, the tiles of list g (first, one past last) that hold a key at or before the
    block's last position; (0, 0) otherwise.  ``attended(i_class, g, entry_mask)``: inside list g a row of class c
    attends an entry iff g is the lowest group the two share.
    """
    mq_h = np.asarray(mq_h, np.uint32); mk_h = np.asarray(mk_h, np.uint32)
    perm, cls_q, cnt_q = class_sort(mq_h)
    seg_q = np.zeros(len(cls_q) + 1, np.int64)
    seg_q[1:] = np.cumsum((cnt_q + pad_q - 1) // pad_q * pad_q)
    perm_q = np.full(int(seg_q[-1]), -1, np.int64)
    src = 0
    for c in range(len(cls_q)):
        perm_q[seg_q[c]:seg_q[c] + cnt_q[c]] = perm[src:src + cnt_q[c]]
        src += cnt_q[c]
    lists = [np.nonzero((mk_h >> g) & 1)[0].astype(np.int64) for g in range(K)]
    cnt_k = np.array([len(l) for l in lists], np.int64)
    seg_k = np.zeros(K + 1, np.int64)
    seg_k[1:] = np.cumsum((cnt_k + pad_k - 1) // pad_k * pad_k)
    perm_k = np.full(int(seg_k[-1]), np.iinfo(np.int32).max, np.int64)
    for g in range(K):
        perm_k[seg_k[g]:seg_k[g] + cnt_k[g]] = lists[g]
    ntile = len(perm_k) // tile
    gbits = np.zeros((ntile, K, tile), bool)
    real = perm_k < len(mk_h)
    member = np.zeros((len(perm_k), K), bool)
    member[real] = ((mk_h[perm_k[real]][:, None] >> np.arange(K)[None, :]) & 1).astype(bool)
    gbits[:] = member.reshape(ntile, tile, K).transpose(0, 2, 1)
    nblk = int(seg_q[-1]) // pad_q
    ranges = np.zeros((nblk, K, 2), np.int64)
    for blk in range(nblk):
        rows = perm_q[blk * pad_q:(blk + 1) * pad_q]
        rows = rows[rows >= 0]
        jq = int(np.searchsorted(seg_q, blk * pad_q, side="right")) - 1
        pmax = int(rows.max())
        for g in range(K):
            if (int(cls_q[jq]) >> g) & 1:
                hi = int(np.count_nonzero(lists[g] <= pmax))
                if hi:
                    ranges[blk, g] = (seg_k[g] // tile, (seg_k[g] + hi - 1) // tile + 1)
    return dict(cls_q=cls_q, cnt_q=cnt_q, seg_q=seg_q, perm_q=perm_q, cnt_k=cnt_k, seg_k=seg_k, perm_k=perm_k,
                gbits=gbits, ranges=ranges)


def assign_hidden(h_bits: np.ndarray, Wg: np.ndarray, C: np.ndarray, topk: int, bias=None):
    """The paper's router.  h_bits uint16 [n, d] (bf16 hidden states), Wg [d, d_g], C [K, d_g], bias [K] or None.

    score[i, g] = <Wg^T h_i, C_g> (+ bias_g), in fp64, in the paper's order (project, then score).  The
    token joins its ``topk`` best groups; exact ties go to the lower group index.
    Returns (masks uint32 [n], margins f64 [n]) with margin = score of the topk-th minus the (topk+1)-th
    group (+inf when topk = K).
    """
    H = bf16_bits_to_f64(np.asarray(h_bits))
    Z = H @ np.asarray(Wg, np.float64)
    S = Z @ np.asarray(C, np.float64).T
    if bias is not None:
        S = S + np.asarray(bias, np.float64)[None, :]
    n, K = S.shape
    order = np.lexsort((np.broadcast_to(np.arange(K), S.shape), -S), axis=1)       # score descending, index ascending
    masks = np.zeros(n, np.uint32)
    for r in range(topk):
        masks |= (np.uint32(1) << order[:, r].astype(np.uint32))
    srt = np.take_along_axis(S, order, axis=1)
    margins = srt[:, topk - 1] - srt[:, topk] if topk < K else np.full(n, np.inf)
    return masks, margins


def router_scores(h_bits: np.ndarray, Wg: np.ndarray, C: np.ndarray) -> np.ndarray:
    """S[i, g] = <Wg^T h_i, C_g> in fp64: project the hidden state, then score it against the centroids."""
    Z = bf16_bits_to_f64(np.asarray(h_bits)) @ np.asarray(Wg, np.float64)
    return Z @ np.asarray(C, np.float64).T


def sinkhorn(S: np.ndarray, tau: float, iters: int) -> np.ndarray:
    """Sinkhorn normalisation of scores S [n, K] at temperature tau: the soft assignments g [n, K].

    Step 1: Q = exp(S / tau).  Step 2, ``iters`` times: divide every column by its sum over the tokens, then
    every row by its sum over the groups.
    """
    Q = np.exp(np.asarray(S, np.float64) / float(tau))
    for _ in range(int(iters)):
        Q = Q / Q.sum(axis=0, keepdims=True)
        Q = Q / Q.sum(axis=1, keepdims=True)
    return Q


def gated_attn(q_bits, k_bits, v_bits, g, lam, window, scale=None, rows=None):
    """Training-time gated attention forward over all causal pairs.

    q_bits uint16 [Hq, n, D], k_bits / v_bits uint16 [Hkv, n, D] (bf16 bit patterns), g float [n, K] (one soft
    assignment per token, shared by all heads), ``lam`` the gate sharpness, ``window`` the local window w.
    For j <= i:  s_ij = scale * <q_i, k_j> * (1 if i - j <= w else sigmoid(lam * <g_i, g_j>)); row softmax.
    Returns (O f64 [Hq, len(rows), D], lse f64 [Hq, len(rows)]); rows default to all.
    """
    Q = bf16_bits_to_f64(np.asarray(q_bits)); Kx = bf16_bits_to_f64(np.asarray(k_bits)); V = bf16_bits_to_f64(np.asarray(v_bits))
    Hq, n, D = Q.shape
    G = Hq // Kx.shape[0]
    sc = 1.0 / np.sqrt(D) if scale is None else float(scale)
    g = np.asarray(g, np.float64)
    rows = np.arange(n) if rows is None else np.asarray(rows, np.int64)
    O = np.zeros((Hq, rows.size, D)); lse = np.zeros((Hq, rows.size))
    j = np.arange(n)
    for r, i in enumerate(rows):
        aff = g @ g[i]                                          # g_i . g_j for every j
        local = (i - j) <= window
        factor = np.where(local, 1.0, 1.0 / (1.0 + np.exp(-float(lam) * aff)))
        causal = j <= i
        for h in range(Hq):
            s = sc * (Kx[h // G] @ Q[h, i]) * factor
            s = s[causal]
            m = s.max()
            e = np.exp(s - m)
            Z = e.sum()
            O[h, r] = (e / Z) @ V[h // G][causal]
            lse[h, r] = m + np.log(Z)
    return O, lse


def sinkhorn_backward(S: np.ndarray, tau: float, iters: int, dG: np.ndarray) -> np.ndarray:
    """d loss / d S for g = sinkhorn(S, tau, iters), given dG = d loss / d g  ([n, K] both).

    Forward steps kept on a tape: Q0 = exp(S / tau); per iteration Y = X / colsum(X), then Z = Y / rowsum(Y).  For a
    division by the sum over an axis, Z = X / sum(X):  dX = (dZ - sum(dZ * Z)) / sum(X) along that axis.
    """
    tau = float(tau)
    X = np.exp(np.asarray(S, np.float64) / tau)
    Q0 = X
    tape = []
    for _ in range(int(iters)):
        c = X.sum(axis=0, keepdims=True); Y = X / c
        r = Y.sum(axis=1, keepdims=True); Z = Y / r
        tape.append((c, Y, r, Z))
        X = Z
    d = np.asarray(dG, np.float64).copy()
    for c, Y, r, Z in reversed(tape):
        d = (d - (d * Z).sum(axis=1, keepdims=True)) / r          # through the division by the row sums
        d = (d - (d * Y).sum(axis=0, keepdims=True)) / c          # through the division by the column sums
    return d * Q0 / tau


def gated_attn_backward(q_bits, k_bits, v_bits, g, lam, window, dO, scale=None):
    """Derivatives of ``gated_attn`` (all rows) with respect to Q, K, V and the soft assignments g.

    dO float [Hq, n, D] = d loss / d O.  With p the row softmax of s_ij = scale * <q_i, k_j> * f_ij over j <= i,
    f_ij = 1 inside the window and sigmoid(lam * <g_i, g_j>) beyond it:
        dV_j += p_ij dO_i;   ds_ij = p_ij (<dO_i, v_j> - <dO_i, o_i>);
        dq_i += ds_ij scale f_ij k_j;   dk_j += ds_ij scale f_ij q_i;
        beyond the window: du_ij = ds_ij scale <q_i, k_j> f_ij (1 - f_ij) lam;   dg_i += du_ij g_j;   dg_j += du_ij g_i.
    Query heads that share a KV head add into the same dK / dV rows; every head adds into dg.
    Returns (dQ [Hq, n, D], dK [Hkv, n, D], dV [Hkv, n, D], dg [n, K]) in fp64.
    """
    Q = bf16_bits_to_f64(np.asarray(q_bits)); Kx = bf16_bits_to_f64(np.asarray(k_bits)); V = bf16_bits_to_f64(np.asarray(v_bits))
    Hq, n, D = Q.shape
    G = Hq // Kx.shape[0]
    sc = 1.0 / np.sqrt(D) if scale is None else float(scale)
    g = np.asarray(g, np.float64); dO = np.asarray(dO, np.float64); lam = float(lam)
    dQ = np.zeros_like(Q); dK = np.zeros_like(Kx); dV = np.zeros_like(V); dg = np.zeros_like(g)
    for i in range(n):
        j = np.arange(i + 1)
        aff = g[:i + 1] @ g[i]
        far = (i - j) > window
        f = np.where(far, 1.0 / (1.0 + np.exp(-lam * aff)), 1.0)
        for h in range(Hq):
            hk = h // G
            qk = Kx[hk, :i + 1] @ Q[h, i]
            s = sc * qk * f
            e = np.exp(s - s.max())
            p = e / e.sum()
            o = p @ V[hk, :i + 1]
            dV[hk, :i + 1] += p[:, None] * dO[h, i][None, :]
            ds = p * (V[hk, :i + 1] @ dO[h, i] - dO[h, i] @ o)
            dQ[h, i] += (ds * sc * f) @ Kx[hk, :i + 1]
            dK[hk, :i + 1] += (ds * sc * f)[:, None] * Q[h, i][None, :]
            du = np.where(far, ds * sc * qk * f * (1.0 - f) * lam, 0.0)
            dg[i] += du @ g[:i + 1]
            dg[:i + 1] += du[:, None] * g[i][None, :]
    return dQ, dK, dV, dg
