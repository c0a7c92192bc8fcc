"""Pins for the CPU oracle: each test ties an oracle function to something other than itself --
an explicit dense-mask brute force, a library routine (torch SDPA / cosine_similarity / topk),
a closed form, a value printed in the paper, or a case worked by hand."""
import math
import os
from math import comb

import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits(x):
    """float array -> bf16 bit patterns (RNE) via torch."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def rand_bits(rng, shape):
    return bits(rng.standard_normal(shape))


def rand_masks(rng, H, n, K, t):
    """uniform random t-subsets of K groups as bit masks"""
    out = np.zeros((H, n), np.uint32)
    for h in range(H):
        for i in range(n):
            out[h, i] = sum(1 << int(g) for g in rng.choice(K, size=t, replace=False))
    return out


def sdpa_causal(qb, kb, vb, scale):
    """library reference: torch scaled_dot_product_attention, causal, fp64, GQA by repeating KV heads"""
    Q = torch.from_numpy(fo.bf16_bits_to_f64(qb)); K = torch.from_numpy(fo.bf16_bits_to_f64(kb))
    V = torch.from_numpy(fo.bf16_bits_to_f64(vb))
    G = Q.shape[0] // K.shape[0]
    K = K.repeat_interleave(G, dim=0); V = V.repeat_interleave(G, dim=0)
    return torch.nn.functional.scaled_dot_product_attention(Q, K, V, is_causal=True, scale=scale).numpy()


# ------------------------------------------------------------------------------------------------
# attention rows
# ------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("n", [1, 2, 3, 17, 64, 129, 257])
@pytest.mark.parametrize("Hq,Hkv,D", [(2, 2, 8), (4, 2, 16), (6, 2, 64)])
def test_rows_vs_dense_bruteforce(n, Hq, Hkv, D):
    """explicit n x n mask + textbook softmax (numpy) == row-by-row C oracle"""
    rng = np.random.default_rng(n * 131 + Hq * 7 + D)
    K = int(rng.choice([2, 4, 8])); t = int(rng.integers(1, K + 1)); w = int(rng.integers(0, n + 2))
    softcap = float(rng.choice([0.0, 3.0]))
    q = rand_bits(rng, (Hq, n, D)); k = rand_bits(rng, (Hkv, n, D)); v = rand_bits(rng, (Hkv, n, D))
    mq = rand_masks(rng, Hq, n, K, t); mk = rand_masks(rng, Hkv, n, K, t)
    r = fo.attn_rows(q, k, v, mq, mk, w, softcap=softcap)
    O, L = fo.dense_brute(q, k, v, mq, mk, w, softcap=softcap)
    np.testing.assert_allclose(r["O"].reshape(Hq, n, D), O, rtol=0, atol=1e-12)
    np.testing.assert_allclose(r["lse"].reshape(Hq, n), L, rtol=0, atol=1e-12)
    # kept counter against the explicit matrix
    G = Hq // Hkv
    cnt = np.stack([fo.kept_matrix(mq[h], mk[h // G], w).sum(axis=1) for h in range(Hq)])
    assert np.array_equal(r["kept"].reshape(Hq, n), cnt)


@pytest.mark.parametrize("Hq,Hkv", [(3, 3), (8, 2)])
def test_window_covers_sequence_is_plain_causal(Hq, Hkv):
    """w >= n: every causal pair is local, so the result is textbook causal attention (torch SDPA),
    whatever the masks say.  With GQA this also pins 'consecutive query heads share a KV head'."""
    rng = np.random.default_rng(5)
    n, D = 96, 32
    q = rand_bits(rng, (Hq, n, D)); k = rand_bits(rng, (Hkv, n, D)); v = rand_bits(rng, (Hkv, n, D))
    mq = rand_masks(rng, Hq, n, 4, 1); mk = rand_masks(rng, Hkv, n, 4, 1)
    ref = sdpa_causal(q, k, v, 1.0 / math.sqrt(D))
    for w in (n, n + 7, 10 * n):
        r = fo.attn_rows(q, k, v, mq, mk, w)
        np.testing.assert_allclose(r["O"].reshape(Hq, n, D), ref, rtol=0, atol=1e-12)


def test_single_group_is_plain_causal():
    """K = 1: assignment puts every token in group 0, every pair shares it -> full causal attention"""
    rng = np.random.default_rng(6)
    Hq, Hkv, n, D = 4, 2, 80, 16
    q = rand_bits(rng, (Hq, n, D)); k = rand_bits(rng, (Hkv, n, D)); v = rand_bits(rng, (Hkv, n, D))
    C = rng.standard_normal((Hkv, 1, D)).astype(np.float32)
    mq, _ = fo.assign(q, C, 1); mk, _ = fo.assign(k, C, 1)
    assert (mq == 1).all() and (mk == 1).all()
    r = fo.attn_rows(q, k, v, mq, mk, 0)
    np.testing.assert_allclose(r["O"].reshape(Hq, n, D), sdpa_causal(q, k, v, 1.0 / math.sqrt(D)), atol=1e-12)


@pytest.mark.parametrize("K,t", [(4, 3), (4, 4), (8, 5), (2, 2)])
def test_pigeonhole_topk_is_plain_causal(K, t):
    """2t > K: any two t-subsets intersect, so nothing is pruned.  The paper's top-k table prints 100 %
    pairs retained for k = 3 and k = 4 of K = 4."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "paper_topk_table.txt")) if not l.startswith("#")]
    for model, k, _, pct in rows:
        if int(k) >= 3:
            assert int(pct) == 100
    rng = np.random.default_rng(K * 10 + t)
    Hq = Hkv = 2; n = 70; D = 8
    q = rand_bits(rng, (Hq, n, D)); k = rand_bits(rng, (Hkv, n, D)); v = rand_bits(rng, (Hkv, n, D))
    mq = rand_masks(rng, Hq, n, K, t); mk = rand_masks(rng, Hkv, n, K, t)
    r = fo.attn_rows(q, k, v, mq, mk, 0)
    np.testing.assert_allclose(r["O"].reshape(Hq, n, D), sdpa_causal(q, k, v, 1.0 / math.sqrt(D)), atol=1e-12)
    assert np.array_equal(fo.kept_pairs(mq, mk, 0), np.full(Hq, n * (n + 1) // 2))


def test_rows_are_stochastic_and_lse_is_log_partition():
    rng = np.random.default_rng(8)
    Hq, Hkv, n, D = 4, 2, 150, 16
    q = rand_bits(rng, (Hq, n, D)); k = rand_bits(rng, (Hkv, n, D)); v = rand_bits(rng, (Hkv, n, D))
    mq = rand_masks(rng, Hq, n, 4, 2); mk = rand_masks(rng, Hkv, n, 4, 2)
    r = fo.attn_rows(q, k, v, mq, mk, 9)
    np.testing.assert_allclose(r["psum"], 1.0, atol=1e-12)
    # V = all-ones -> every output coordinate equals the total weight 1
    ones = bits(np.ones((Hkv, n, D)))
    r1 = fo.attn_rows(q, k, ones, mq, mk, 9)
    np.testing.assert_allclose(r1["O"], 1.0, atol=1e-12)
    # exp(lse) is the unnormalised partition sum: check through torch.logsumexp on the kept logits
    Q = fo.bf16_bits_to_f64(q); Kd = fo.bf16_bits_to_f64(k)
    for (h, i) in [(0, 0), (1, 37), (3, 149)]:
        keep = fo.kept_matrix(mq[h], mk[h // 2], 9)[i]
        s = (Q[h, i] @ Kd[h // 2].T) / math.sqrt(D)
        ref = torch.logsumexp(torch.from_numpy(s[keep]), 0).item()
        assert abs(r["lse"][h * n + i] - ref) < 1e-12


def test_hand_worked_case():
    """n=4, D=2, K=2 groups, top-1, w=1, scale=1; everything below is worked by hand.

    centroids c0=(1,0), c1=(0,1).  x0=(1,0)->g0, x1=(0,1)->g1, x2=(0,2)->g1, x3=(2,0)->g0 (Q = K = x).
    kept sets: row0 {0}; row1 {0 (local), 1}; row2 {1 (local), 2}  (0 is 2 away and in another group);
    row3 {0 (far, same group), 2 (local, other group), 3}  (1 is 2 away and in another group).
    """
    x = np.array([[1, 0], [0, 1], [0, 2], [2, 0]], np.float32)[None]
    V = np.array([[1, 0], [0, 1], [1, 1], [-1, 2]], np.float32)[None]
    C = np.array([[[1, 0], [0, 1]]], np.float32)
    m, margins = fo.assign(bits(x), C, 1)
    assert m.tolist() == [[1, 2, 2, 1]]
    np.testing.assert_allclose(margins, 1.0, atol=1e-15)        # cosines are exactly 1 and 0
    r = fo.attn_rows(bits(x), bits(x), bits(V), m, m, 1, scale=1.0)
    e = math.exp
    O = r["O"]; L = r["lse"]
    assert r["kept"].tolist() == [1, 2, 2, 3]
    np.testing.assert_allclose(O[0], [1, 0], atol=1e-15); assert abs(L[0] - 1.0) < 1e-15
    # row1: s10 = 0, s11 = 1
    np.testing.assert_allclose(O[1], [1 / (1 + e(1)), e(1) / (1 + e(1))], atol=1e-15)
    assert abs(L[1] - math.log(1 + e(1))) < 1e-15
    # row2: s21 = 2, s22 = 4
    z = e(2) + e(4)
    np.testing.assert_allclose(O[2], [e(4) / z, (e(2) + e(4)) / z], atol=1e-15)
    assert abs(L[2] - math.log(z)) < 1e-14
    # row3: s30 = 2, s32 = 0, s33 = 4
    z = e(2) + 1 + e(4)
    np.testing.assert_allclose(O[3], [(e(2) + 1 - e(4)) / z, (1 + 2 * e(4)) / z], atol=1e-15)
    assert abs(L[3] - math.log(z)) < 1e-14
    # w = 0 drops the distance-1 neighbours of other groups; w = 2 brings back (2,0) and (3,1)
    assert fo.attn_rows(bits(x), bits(x), bits(V), m, m, 0, scale=1.0)["kept"].tolist() == [1, 1, 2, 2]
    assert fo.attn_rows(bits(x), bits(x), bits(V), m, m, 2, scale=1.0)["kept"].tolist() == [1, 2, 3, 4]


def test_softcap_closed_form_and_limit():
    """two keys: weight ratio is exp(c*tanh(s1/c) - c*tanh(s0/c)); a huge cap changes nothing"""
    q = np.array([[[0, 0], [3, 1]]], np.float32); k = np.array([[[2, 0], [1, 3]]], np.float32)
    v = np.array([[[1, 0], [0, 1]]], np.float32)
    m = np.ones((1, 2), np.uint32)
    c = 2.0
    r = fo.attn_rows(bits(q), bits(k), bits(v), m, m, 5, scale=0.5, softcap=c)
    s0 = c * math.tanh(0.5 * 6 / c); s1 = c * math.tanh(0.5 * 6 / c)
    assert s0 == s1
    np.testing.assert_allclose(r["O"][1], [0.5, 0.5], atol=1e-15)
    k2 = np.array([[[2, 0], [1, 1]]], np.float32)                 # s0 = 3, s1 = 2 before capping
    r = fo.attn_rows(bits(q), bits(k2), bits(v), m, m, 5, scale=0.5, softcap=c)
    a, b = c * math.tanh(3 / c), c * math.tanh(2 / c)
    np.testing.assert_allclose(r["O"][1], [math.exp(a) / (math.exp(a) + math.exp(b)),
                                           math.exp(b) / (math.exp(a) + math.exp(b))], atol=1e-15)
    assert abs(r["lse"][1] - math.log(math.exp(a) + math.exp(b))) < 1e-15
    rng = np.random.default_rng(3)
    qq = rand_bits(rng, (2, 40, 8)); kk = rand_bits(rng, (2, 40, 8)); vv = rand_bits(rng, (2, 40, 8))
    mm = rand_masks(rng, 2, 40, 4, 2)
    big = fo.attn_rows(qq, kk, vv, mm, mm, 4, softcap=1e9)["O"]
    off = fo.attn_rows(qq, kk, vv, mm, mm, 4, softcap=0.0)["O"]
    np.testing.assert_allclose(big, off, atol=1e-9)


def test_two_set_merge_matches_and_double_count_fails():
    """Appendix D: sets A (same-group causal) and B (cross-group local) merged through their
    logsumexps equal the masked definition (the paper reports cosine similarity 1.0000); the
    overlapping same-group + all-local split double counts and must NOT match."""
    rng = np.random.default_rng(11)
    n, D, K, w = 200, 16, 4, 12
    q = rand_bits(rng, (n, D)); k = rand_bits(rng, (n, D)); v = rand_bits(rng, (n, D))
    g = rng.integers(0, K, n)
    m = (1 << g).astype(np.uint32)[None]
    ref = fo.attn_rows(q[None], k[None], v[None], m, m, w)
    O, L = fo.ab_merge(q, k, v, g, w)
    np.testing.assert_allclose(O, ref["O"], atol=1e-12)
    np.testing.assert_allclose(L, ref["lse"], atol=1e-12)

    def cos(a, b):
        return float((a * b).sum() / np.sqrt((a * a).sum() * (b * b).sum()))

    assert round(cos(O, ref["O"]), 4) == 1.0
    Obad, _ = fo.ab_merge(q, k, v, g, w, double_count=True)
    assert np.abs(Obad - ref["O"]).max() > 1e-2
    assert cos(Obad, ref["O"]) < 0.9999


# ------------------------------------------------------------------------------------------------
# kept-pair counts
# ------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("n,w", [(1, 0), (33, 0), (130, 7), (257, 300)])
def test_kept_pairs_vs_explicit_matrix(n, w):
    rng = np.random.default_rng(n + w)
    Hq, Hkv = 4, 2
    mq = rand_masks(rng, Hq, n, 8, 2); mk = rand_masks(rng, Hkv, n, 8, 2)
    want = [int(fo.kept_matrix(mq[h], mk[h // 2], w).sum()) for h in range(Hq)]
    assert fo.kept_pairs(mq, mk, w).tolist() == want


@pytest.mark.parametrize("K,t", [(4, 1), (4, 2), (8, 2), (8, 1)])
def test_far_kept_fraction_closed_form(K, t):
    """independent uniform t-subsets share a group with probability 1 - C(K-t,t)/C(K,t); for t = 1
    this is the paper's 1/K (n^2/K cost; 25-26 % of pairs retained at K=4, k=1 in its top-k table)."""
    if t == 1:
        model = {int(l.split()[0]): float(l.split()[1])
                 for l in open(os.path.join(GOLDEN, "paper_speedup_model.txt")) if not l.startswith("#")}
        assert abs(model[K] - (1 - comb(K - t, t) / comb(K, t))) < 1e-15
    if (K, t) == (4, 1):
        tab = [l.split() for l in open(os.path.join(GOLDEN, "paper_topk_table.txt")) if not l.startswith("#")]
        assert all(abs(int(p) - 25) <= 1 for _, k, _, p in tab if int(k) == 1)
    rng = np.random.default_rng(K * 100 + t)
    n = 3000
    mq = rand_masks(rng, 1, n, K, t); mk = rand_masks(rng, 1, n, K, t)
    far_total = n * (n + 1) // 2 - n                          # w = 0: only the diagonal is local
    frac = (int(fo.kept_pairs(mq, mk, 0)[0]) - n) / far_total
    want = 1 - comb(K - t, t) / comb(K, t)
    assert abs(frac - want) < 4 * math.sqrt(want * (1 - want) / n)   # rows are the independent units


# ------------------------------------------------------------------------------------------------
# assignment
# ------------------------------------------------------------------------------------------------

def test_assign_matches_library_cosine_topk():
    """torch cosine_similarity + topk in fp64 as the library reference (no exact ties in random data)"""
    rng = np.random.default_rng(21)
    H, Hkv, n, D, K, t = 6, 3, 300, 32, 8, 3
    x = rand_bits(rng, (H, n, D))
    C = rng.standard_normal((Hkv, K, D)).astype(np.float32) * rng.uniform(0.5, 3, (Hkv, K, 1)).astype(np.float32)
    masks, margins = fo.assign(x, C, t)
    X = torch.from_numpy(fo.bf16_bits_to_f64(x))
    Ct = torch.from_numpy(C.astype(np.float64)).repeat_interleave(H // Hkv, dim=0)      # [H, K, D]
    cs = torch.nn.functional.cosine_similarity(X[:, :, None, :], Ct[:, None, :, :], dim=-1, eps=0)
    top = torch.topk(cs, t + 1, dim=-1)
    want = (1 << top.indices[..., :t]).sum(-1).numpy().astype(np.uint32)
    assert np.array_equal(masks, want)
    np.testing.assert_allclose(margins, (top.values[..., t - 1] - top.values[..., t]).numpy(), atol=1e-14)


def test_assign_geometry_ties_scaling():
    # D = 2, centroids at 0, 90, 180 degrees (non-unit lengths: cosine ignores them)
    C = np.array([[[3, 0], [0, 0.5], [-2, 0]]], np.float32)
    ang = np.deg2rad([10, 80, 100, 170, 44, 46])
    x = np.stack([np.cos(ang), np.sin(ang)], 1).astype(np.float32)[None] * 4
    m, mg = fo.assign(bits(x), C, 1)
    assert m.tolist() == [[1, 2, 2, 4, 1, 2]]
    m2, _ = fo.assign(bits(x), C, 2)
    assert m2.tolist() == [[3, 3, 6, 6, 3, 3]]
    # margin for the 10-degree vector at t=1: cos(10deg) - cos(80deg), up to bf16 rounding of x
    xb = fo.bf16_bits_to_f64(bits(x))[0, 0]
    a = math.atan2(xb[1], xb[0])
    assert abs(mg[0, 0] - (math.cos(a) - math.cos(math.pi / 2 - a))) < 1e-12
    # exact ties: duplicate centroids -> lower index wins; zero vector -> groups 0..t-1
    Cd = np.array([[[1, 1], [1, 1], [1, 1], [-1, 0]]], np.float32)
    z = np.array([[[2, 2], [0, 0], [-1, 0]]], np.float32)
    m, mg = fo.assign(bits(z), Cd, 2)
    assert m.tolist() == [[0b0011, 0b0011, 0b1001]]
    assert mg[0, 0] == 0.0 and mg[0, 1] == 0.0
    # positive rescaling of tokens (exact in bf16) and of centroids changes nothing; t = K margin is inf
    rng = np.random.default_rng(2)
    xr = rng.standard_normal((2, 50, 16)).astype(np.float32)
    Cr = rng.standard_normal((2, 4, 16)).astype(np.float32)
    a, _ = fo.assign(bits(xr), Cr, 2)
    b, _ = fo.assign(bits(bits_scale(xr, 4.0)), Cr * np.float32(0.125), 2)
    assert np.array_equal(a, b)
    full, mg = fo.assign(bits(xr), Cr, 4)
    assert (full == 15).all() and np.isinf(mg).all()


def bits_scale(x, s):
    return fo.bf16_bits_to_f64(bits(x)).astype(np.float32) * np.float32(s)


def test_assign_dominant_centroid():
    """x = 5*c_g + small noise must land in group g first"""
    rng = np.random.default_rng(4)
    Hkv, K, D = 2, 8, 64
    C = rng.standard_normal((Hkv, K, D)).astype(np.float32)
    C /= np.linalg.norm(C, axis=-1, keepdims=True)
    g = rng.integers(0, K, (4, 100))
    x = 5 * C[np.arange(4)[:, None] // 2, g] + 0.1 * rng.standard_normal((4, 100, D)).astype(np.float32)
    m, _ = fo.assign(bits(x), C, 1)
    assert np.array_equal(m, (1 << g).astype(np.uint32))


# ------------------------------------------------------------------------------------------------
# tile summaries and class sort
# ------------------------------------------------------------------------------------------------

def test_tile_reference_is_sound_and_tight():
    """a far tile pair is dead exactly when the explicit mask has no kept pair in it (given w), and
    'full' tiles are entirely kept"""
    rng = np.random.default_rng(31)
    Hq, Hkv, n, BM, BN, w = 2, 1, 200, 16, 8, 10
    # few groups per tile so that some tiles really die: group depends on position block
    blk = (np.arange(n) // 24) % 4
    mk = (1 << blk).astype(np.uint32)[None]
    mq = np.stack([(1 << blk), (1 << ((blk + (np.arange(n) % 7 == 0)) % 4))]).astype(np.uint32)
    ref = fo.tile_reference(mq, mk, w, BM, BN)
    nqt, nkt = ref["far"].shape
    dead_seen = live_seen = full_seen = 0
    for h in range(Hq):
        M = fo.kept_matrix(mq[h], mk[0], w)
        for a in range(nqt):
            for b in range(nkt):
                rows = slice(a * BM, min(n, (a + 1) * BM)); cols = slice(b * BN, min(n, (b + 1) * BN))
                sub = M[rows, cols]
                i = np.arange(n)[rows][:, None]; j = np.arange(n)[cols][None, :]
                is_far = bool(((i - j) > w).all())
                assert ref["far"][a, b] == is_far
                if is_far and not ref["live"][h, a, b]:
                    assert not sub.any(); dead_seen += 1
                if ref["live"][h, a, b]:
                    live_seen += 1
                if ref["full"][h, a, b]:
                    assert sub.all() and ref["live"][h, a, b]; full_seen += 1
    assert dead_seen > 0 and live_seen > 0 and full_seen > 0


def test_class_sort_is_stable_and_preserves_kept_sets():
    """sorting tokens by mask value with a stable sort keeps positions ascending inside a class, and
    the kept rule evaluated on (sorted index -> original position) is the same set of pairs"""
    rng = np.random.default_rng(41)
    n, w = 300, 9
    mq = rand_masks(rng, 1, n, 4, 2)[0]; mk = rand_masks(rng, 1, n, 4, 2)[0]
    pq, cq, nq = fo.class_sort(mq); pk, ck, nk = fo.class_sort(mk)
    assert sorted(pq.tolist()) == list(range(n)) and nq.sum() == n
    off = 0
    for c, cnt in zip(cq, nq):
        seg = pq[off:off + cnt]
        assert (mq[seg] == c).all() and (np.diff(seg) > 0).all()
        off += cnt
    M = fo.kept_matrix(mq, mk, w)
    posq = pq[:, None]; posk = pk[None, :]
    share = (mq[pq][:, None] & mk[pk][None, :]) != 0
    Ms = (posk <= posq) & (((posq - posk) <= w) | share)
    assert np.array_equal(Ms, M[np.ix_(pq, pk)])


@pytest.mark.parametrize("n,K,t", [(700, 4, 2), (900, 8, 2), (600, 6, 3), (500, 4, 1), (300, 5, 5)])
def test_group_major_lists_cover_every_sharing_pair_exactly_once(n, K, t):
    """walking, for every query, the lists of its own groups up to its position and attending an entry only under the
    lowest shared group visits each causal pair with intersecting masks exactly once and no other pair; the listed
    tile ranges contain all of them and end on a tile that holds one"""
    rng = np.random.default_rng(n + K + t)
    mq = np.array([sum(1 << int(g) for g in rng.choice(K, t, replace=False)) for _ in range(n)], np.uint32)
    mk = np.array([sum(1 << int(g) for g in rng.choice(K, t, replace=False)) for _ in range(n)], np.uint32)
    L = fo.group_major_layout(mq, mk, K)
    share = ((mq[:, None] & mk[None, :]) != 0) & (np.arange(n)[None, :] <= np.arange(n)[:, None])     # explicit matrix
    times = np.zeros((n, n), np.int64)
    in_range = np.zeros((n, n), bool)
    for blk in range(L["ranges"].shape[0]):
        rows = L["perm_q"][blk * 256:(blk + 1) * 256]
        rows = rows[rows >= 0]
        jq = int(np.searchsorted(L["seg_q"], blk * 256, side="right")) - 1
        assert (mq[rows] == L["cls_q"][jq]).all()
        for g in range(K):
            first, last = L["ranges"][blk, g]
            if not (int(L["cls_q"][jq]) >> g) & 1:
                assert first == last == 0
                continue
            if last > first:
                assert first * 128 == L["seg_k"][g] and last * 128 <= L["seg_k"][g + 1]
            slots = np.arange(first * 128, last * 128)
            pos = L["perm_k"][slots]
            real = pos < n
            lower = int(L["cls_q"][jq]) & ((1 << g) - 1)
            ent_mask = np.zeros(len(slots), np.int64)
            ent_mask[real] = mk[pos[real]]
            assert ((ent_mask[real] >> g) & 1).all()                       # the list holds members of g only
            assert (np.diff(pos[real]) > 0).all()                          # in token order
            ok_col = real & ((ent_mask & lower) == 0)                      # not attended under a lower shared group
            for i in rows:
                cols = pos[ok_col & (pos <= i)]
                np.add.at(times[i], cols, 1)
                in_range[i, pos[real & (pos <= i)]] = True
            if last > first:                                               # the last listed tile holds a causal key of the block
                assert (pos[(last - first - 1) * 128:][real[(last - first - 1) * 128:]] <= rows.max()).any()
    assert np.array_equal(times, share.astype(np.int64))
    # gbits is the membership of every list entry
    flat = L["gbits"].transpose(0, 2, 1).reshape(-1, K)
    real = L["perm_k"] < n
    want = ((mk[L["perm_k"][real]][:, None] >> np.arange(K)[None, :]) & 1).astype(bool)
    assert np.array_equal(flat[real], want) and not flat[~real].any()


@pytest.mark.parametrize("n,K,t,w", [(700, 4, 2, 40), (1500, 4, 1, 100), (900, 8, 2, 0), (600, 2, 1, 1000)])
def test_sorted_layout_ranges_cover_exactly_the_tiles_with_kept_pairs(n, K, t, w):
    """every kept pair of the explicit mask lies in a listed tile of its key class; the first and last listed
    tile of a sharing class hold a kept pair; listed tiles of a non-sharing class touch the window span"""
    rng = np.random.default_rng(n + K)
    mq = np.array([sum(1 << int(g) for g in rng.choice(K, t, replace=False)) for _ in range(n)], np.uint32)
    mk = np.array([sum(1 << int(g) for g in rng.choice(K, t, replace=False)) for _ in range(n)], np.uint32)
    L = fo.sorted_layout(mq, mk, w)
    kept = fo.kept_matrix(mq, mk, w)
    # permutations are stable class sorts
    for perm, cls, cnt, seg, m in ((L["perm_q"], L["cls_q"], L["cnt_q"], L["seg_q"], mq),
                                   (L["perm_k"], L["cls_k"], L["cnt_k"], L["seg_k"], mk)):
        real = perm[(perm >= 0) & (perm < n)]
        assert sorted(real.tolist()) == list(range(n))
        for c in range(len(cls)):
            part = perm[seg[c]:seg[c] + cnt[c]]
            assert (m[part] == cls[c]).all() and (np.diff(part) > 0).all()
    slot_of_key = np.empty(n, np.int64)
    valid_k = np.nonzero(L["perm_k"] < n)[0]
    slot_of_key[L["perm_k"][valid_k]] = valid_k
    cls_of_tile = np.searchsorted(L["seg_k"], np.arange(len(L["perm_k"]) // 128) * 128, side="right") - 1
    for blk in range(L["ranges"].shape[0]):
        rows = L["perm_q"][blk * 256:(blk + 1) * 256]
        rows = rows[rows >= 0]
        keys = np.nonzero(kept[rows].any(axis=0))[0]
        tiles = np.unique(slot_of_key[keys] // 128)
        for tl in tiles:
            first, last = L["ranges"][blk, cls_of_tile[tl]]
            assert first <= tl < last
        jq = int(np.searchsorted(L["seg_q"], blk * 256, side="right")) - 1
        for jk in range(len(L["cls_k"])):
            first, last = L["ranges"][blk, jk]
            if last > first and int(L["cls_q"][jq]) & int(L["cls_k"][jk]):
                assert first in tiles and last - 1 in tiles
            if last > first:
                assert first * 128 >= L["seg_k"][jk] and last * 128 <= L["seg_k"][jk + 1]


def _bf16_bits(x):
    return torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def test_assign_hidden_matches_torch_topk_and_reduces_to_cosine_assign():
    rng = np.random.default_rng(5)
    n, d, dg, K, t = 400, 96, 16, 6, 2
    hb = _bf16_bits(rng.standard_normal((n, d)))
    W = rng.standard_normal((d, dg)); C = rng.standard_normal((K, dg)); b = rng.standard_normal(K)
    masks, margins = fo.assign_hidden(hb, W, C, t, bias=b)
    H = torch.from_numpy(hb.view(np.int16)).view(torch.bfloat16).double()
    S = (H @ torch.from_numpy(W)) @ torch.from_numpy(C).T + torch.from_numpy(b)
    idx = torch.topk(S, t, dim=1).indices.numpy()
    ref = np.zeros(n, np.uint32)
    for r in range(t):
        ref |= np.uint32(1) << idx[:, r].astype(np.uint32)
    assert np.array_equal(masks, ref) and (margins > 0).all()
    # W = identity, unit centroids, no bias: the ranking of dot products is the ranking of cosines
    Cn = rng.standard_normal((K, d)); Cn /= np.linalg.norm(Cn, axis=1, keepdims=True)
    m_hidden, _ = fo.assign_hidden(hb, np.eye(d), Cn, t)
    m_cos, _ = fo.assign(hb[None], Cn[None].astype(np.float32), t)
    m_hidden32, _ = fo.assign_hidden(hb, np.eye(d), Cn.astype(np.float32), t)
    assert np.array_equal(m_hidden32, m_cos[0])
    # ties go to the lower index; a dominant bias always wins
    m_tie, mg = fo.assign_hidden(hb[:5], np.zeros((d, dg)), C, 2)
    assert (m_tie == 0b11).all() and (mg == 0).all()
    m_bias, _ = fo.assign_hidden(hb, W, C, 1, bias=np.array([0, 0, 0, 1e9, 0, 0.0]))
    assert (m_bias == 1 << 3).all()


def test_bias_is_the_inference_residue_of_sinkhorn_column_scaling():
    """Sec. 2: Q <- exp(S/tau); N times: divide by the sum over tokens, then by the sum over groups.  The result is
    diag(r) exp(S/tau) diag(c), so every row ranks its groups like S + tau log c: with bias = tau log c the router
    reproduces the balanced assignment's top-k."""
    rng = np.random.default_rng(9)
    n, d, dg, K, tau = 300, 64, 16, 4, 0.7
    hb = _bf16_bits(rng.standard_normal((n, d)))
    W = rng.standard_normal((d, dg)) * 0.05; C = rng.standard_normal((K, dg)); C[0] *= 3.0      # group 0 would dominate
    S = (fo.bf16_bits_to_f64(hb) @ W) @ C.T
    Q = np.exp(S / tau)
    logc = np.zeros(K)
    for _ in range(10):
        col = Q.sum(axis=0, keepdims=True)
        Q = Q / col; logc -= np.log(col[0])
        Q = Q / Q.sum(axis=1, keepdims=True)
    top_sinkhorn = np.argsort(-Q, axis=1, kind="stable")[:, :2]
    want = (np.uint32(1) << top_sinkhorn[:, 0].astype(np.uint32)) | (np.uint32(1) << top_sinkhorn[:, 1].astype(np.uint32))
    got, _ = fo.assign_hidden(hb, W, C, 2, bias=tau * logc)
    assert np.array_equal(got, want)
    plain, _ = fo.assign_hidden(hb, W, C, 2)
    assert (plain != want).any()            # without the bias the unbalanced ranking differs
    mass = Q.sum(axis=0)                     # Sinkhorn did balance the groups' mass; the plain row softmax does not
    P = np.exp(S / tau); P /= P.sum(axis=1, keepdims=True)
    # (Sinkhorn converges linearly: ten iterations leave these inputs within 5 % of balance, the row softmax is 2x off)
    assert mass.max() / mass.min() < 1.05 < 2.0 < P.sum(axis=0).max() / P.sum(axis=0).min()


# ---------------------------------------------------------------- training-time forward: Sinkhorn and the soft gate (Sec. 2)
def test_router_scores_hand_case():
    """d = 2, d_g = 2, K = 2 in small integers, worked by hand: z = h Wg, S = z C^T"""
    h = bits(np.array([[1., 2.], [3., -1.]]))
    Wg = np.array([[1., 0.], [2., 1.]])            # z_0 = (1 + 4, 2) = (5, 2);  z_1 = (3 - 2, -1) = (1, -1)
    C = np.array([[1., 1.], [0., -2.]])            # S_0 = (7, -4);  S_1 = (0, 2)
    np.testing.assert_array_equal(fo.router_scores(h, Wg, C), np.array([[7., -4.], [0., 2.]]))


def test_sinkhorn_hand_2x2():
    """exp(S / tau) = [[1, 2], [3, 4]]; two iterations worked by hand in fractions.
    It. 1: column sums 4, 6 -> [[1/4, 1/3], [3/4, 2/3]]; row sums 7/12, 17/12 -> [[3/7, 4/7], [9/17, 8/17]].
    It. 2: column sums 114/119, 124/119 -> [[17/38, 17/31], [21/38, 14/31]]; row sums 1173/1178, 1183/1178
           -> [[31/69, 38/69], [93/169, 76/169]]."""
    tau = 0.7
    S = tau * np.log(np.array([[1., 2.], [3., 4.]]))
    np.testing.assert_allclose(fo.sinkhorn(S, tau, 1), [[3 / 7, 4 / 7], [9 / 17, 8 / 17]], rtol=1e-14)
    np.testing.assert_allclose(fo.sinkhorn(S, tau, 2), [[31 / 69, 38 / 69], [93 / 169, 76 / 169]], rtol=1e-14)
    # rows first, columns second (the wrong order) gives [[1/3, 2/3], [3/7, 4/7]] -> columns ... : not the values above
    assert abs(fo.sinkhorn(S, tau, 1)[0, 0] - (1 / 3) / (1 / 3 + 3 / 7)) > 1e-3


def test_sinkhorn_2x2_limit_closed_form():
    """Two tokens, two groups: the doubly stochastic scaling of [[a, b], [c, d]] is [[x, 1-x], [1-x, x]] with
    x = sqrt(ad) / (sqrt(ad) + sqrt(bc)) (diagonal scalings keep the cross ratio ad / bc)."""
    a, b, c, d = 1., 2., 3., 4.
    x = math.sqrt(a * d) / (math.sqrt(a * d) + math.sqrt(b * c))
    got = fo.sinkhorn(np.log(np.array([[a, b], [c, d]])), 1.0, 300)
    np.testing.assert_allclose(got, [[x, 1 - x], [1 - x, x]], rtol=1e-12)


def test_sinkhorn_invariants():
    rng = np.random.default_rng(5)
    n, K, tau = 400, 8, 0.5
    S = rng.standard_normal((n, K))
    g = fo.sinkhorn(S, tau, 10)
    np.testing.assert_allclose(g.sum(axis=1), 1.0, atol=1e-14)           # the last step normalises the rows
    assert np.all(g > 0)
    np.testing.assert_allclose(fo.sinkhorn(S, tau, 200).sum(axis=0), n / K, rtol=1e-9)   # balanced groups at convergence
    # a per-group offset of the scores is removed by the first division over the tokens
    np.testing.assert_allclose(fo.sinkhorn(S + rng.standard_normal(K)[None, :], tau, 10), g, rtol=1e-11)
    # a per-token offset is not (finite number of iterations): the order of the two divisions matters
    assert np.abs(fo.sinkhorn(S + rng.standard_normal(n)[:, None], tau, 1) - fo.sinkhorn(S, tau, 1)).max() > 1e-3
    # one group: everything belongs to it; equal scores: equal shares
    np.testing.assert_array_equal(fo.sinkhorn(S[:, :1], tau, 10), np.ones((n, 1)))
    np.testing.assert_allclose(fo.sinkhorn(np.full((n, K), 0.3), tau, 10), 1.0 / K, rtol=1e-14)
    # one token: the division over tokens makes every entry 1, the division over groups 1/K
    np.testing.assert_allclose(fo.sinkhorn(S[:1], tau, 3), np.full((1, K), 1.0 / K), rtol=1e-14)


def test_gated_attn_hand_case():
    """n = 3, D = 1, K = 2, w = 0, lambda = ln 3, scale = ln 2, worked by hand.
    g = (e0, e1, e0): sigmoid(lambda * 1) = 3/4, sigmoid(0) = 1/2.  q = (1, 1, 2), k = (2, 4, 1), v = (7, 14, 21).
    Row 0: s = 2 ln2 -> o = 7, lse = ln 4.
    Row 1: s_10 = 1*2*ln2 * 1/2 = ln 2 -> 2;  s_11 = 4 ln 2 -> 16;  o = (2*7 + 16*14) / 18 = 119/9, lse = ln 18.
    Row 2: s_20 = 2*2*ln2 * 3/4 = 3 ln 2 -> 8;  s_21 = 2*4*ln2 * 1/2 = 4 ln 2 -> 16;  s_22 = 2 ln 2 -> 4;
           o = (8*7 + 16*14 + 4*21) / 28 = 13, lse = ln 28."""
    q = bits(np.array([[[1.], [1.], [2.]]])); k = bits(np.array([[[2.], [4.], [1.]]])); v = bits(np.array([[[7.], [14.], [21.]]]))
    g = np.array([[1., 0.], [0., 1.], [1., 0.]])
    O, lse = fo.gated_attn(q, k, v, g, math.log(3.0), 0, scale=math.log(2.0))
    np.testing.assert_allclose(O[0, :, 0], [7.0, 119.0 / 9.0, 13.0], rtol=1e-13)
    np.testing.assert_allclose(lse[0], np.log([4.0, 18.0, 28.0]), rtol=1e-13)
    # window 1 makes (1,0) and (2,1) local: row 1 -> (4*7 + 16*14)/20, row 2 -> (8*7 + 256*14 + 4*21)/268
    O, lse = fo.gated_attn(q, k, v, g, math.log(3.0), 1, scale=math.log(2.0))
    np.testing.assert_allclose(O[0, :, 0], [7.0, 252.0 / 20.0, 3724.0 / 268.0], rtol=1e-13)


def test_gated_attn_reduces_to_library_attention():
    rng = np.random.default_rng(11)
    Hq, Hkv, n, D, K = 4, 2, 96, 16, 4
    qb, kb, vb = rand_bits(rng, (Hq, n, D)), rand_bits(rng, (Hkv, n, D)), rand_bits(rng, (Hkv, n, D))
    g = fo.sinkhorn(rng.standard_normal((n, K)), 0.5, 10)
    ref = sdpa_causal(qb, kb, vb, 1.0 / math.sqrt(D))
    # the window covers the whole sequence: the gate never applies
    O, _ = fo.gated_attn(qb, kb, vb, g, 7.0, n, None)
    np.testing.assert_allclose(O, ref, atol=1e-12)
    # every token wholly in one group and a sharp gate: sigmoid(60) = 1 to 1e-26
    one = np.zeros((n, K)); one[:, 2] = 1.0
    O, _ = fo.gated_attn(qb, kb, vb, one, 60.0, 3, None)
    np.testing.assert_allclose(O, ref, atol=1e-12)


def test_gated_attn_half_gate_is_half_scale():
    """g = 0 gives the gate sigmoid(0) = 1/2 on every distant pair.  With w = 0 only the diagonal is local, and
    with k_i orthogonal to q_i the diagonal logit is 0 at any scale: the result is library attention at half
    the scale."""
    rng = np.random.default_rng(12)
    H, n = 3, 64
    q = rng.integers(-4, 5, size=(H, n, 2)).astype(np.float64)
    k = np.stack([-q[..., 1], q[..., 0]], axis=-1) * rng.integers(1, 3, size=(H, n, 1))
    qb, kb, vb = bits(q), bits(k), rand_bits(rng, (H, n, 2))
    O, _ = fo.gated_attn(qb, kb, vb, np.zeros((n, 4)), 5.0, 0, scale=0.25)
    np.testing.assert_allclose(O, sdpa_causal(qb, kb, vb, 0.125), atol=1e-12)


# ---------------------------------------------------------------- derivatives of the training-time forward (Sec. 2)
def test_sinkhorn_backward_matches_finite_differences_and_autograd():
    """the chain rule through the N column / row divisions against central differences of the oracle's own forward and
    against automatic differentiation of the same steps written with torch"""
    import torch
    rng = np.random.default_rng(4)
    n, K, tau, N = 9, 4, 0.7, 3
    S = rng.standard_normal((n, K)) * 0.5
    dG = rng.standard_normal((n, K))
    got = fo.sinkhorn_backward(S, tau, N, dG)
    num = np.zeros_like(S)
    eps = 1e-6
    for a in range(n):
        for b in range(K):
            Sp = S.copy(); Sp[a, b] += eps
            Sm = S.copy(); Sm[a, b] -= eps
            num[a, b] = ((fo.sinkhorn(Sp, tau, N) - fo.sinkhorn(Sm, tau, N)) * dG).sum() / (2 * eps)
    assert np.abs(got - num).max() < 1e-7
    St = torch.tensor(S, dtype=torch.float64, requires_grad=True)
    Qt = torch.exp(St / tau)
    for _ in range(N):
        Qt = Qt / Qt.sum(dim=0, keepdim=True)
        Qt = Qt / Qt.sum(dim=1, keepdim=True)
    assert np.abs(Qt.detach().numpy() - fo.sinkhorn(S, tau, N)).max() < 1e-14
    (Qt * torch.tensor(dG)).sum().backward()
    assert np.abs(got - St.grad.numpy()).max() < 1e-12
    # the assignments do not change when one group's scores are shifted by a constant (the first column division removes
    # it): the gradient summed over the tokens of a column vanishes
    assert np.abs(got.sum(axis=0)).max() < 1e-12


@pytest.mark.parametrize("Hq,Hkv,w", [(2, 1, 1), (2, 2, 0), (4, 2, 3)])
def test_gated_attention_backward_matches_autograd_and_finite_differences(Hq, Hkv, w):
    """dQ, dK, dV and d(assignments) of Eq. 2's forward: automatic differentiation of the explicit dense formula
    (whose forward equals the oracle's), plus central differences of the oracle's forward on a few entries"""
    import torch
    rng = np.random.default_rng(10 * Hq + w)
    n, D, K, lam = 7, 4, 3, 3.0
    bf = lambda x: torch.tensor(x).to(torch.bfloat16)
    Qb, Kb, Vb = bf(rng.standard_normal((Hq, n, D))), bf(rng.standard_normal((Hkv, n, D))), bf(rng.standard_normal((Hkv, n, D)))
    bits = lambda t: t.view(torch.int16).numpy().view(np.uint16)
    g = rng.random((n, K)); g /= g.sum(axis=1, keepdims=True)
    dO = rng.standard_normal((Hq, n, D))
    dQ, dK, dV, dg = fo.gated_attn_backward(bits(Qb), bits(Kb), bits(Vb), g, lam, w, dO)
    # explicit dense formula in torch
    Qt = Qb.double().requires_grad_(True); Kt = Kb.double().requires_grad_(True); Vt = Vb.double().requires_grad_(True)
    gt = torch.tensor(g, requires_grad=True)
    G = Hq // Hkv
    idx = torch.arange(n)
    causal = idx[None, :] <= idx[:, None]
    far = (idx[:, None] - idx[None, :]) > w
    f = torch.where(far, torch.sigmoid(lam * (gt @ gt.T)), torch.ones((), dtype=torch.float64))
    outs = []
    for h in range(Hq):
        s = (Qt[h] @ Kt[h // G].T) / D ** 0.5 * f
        s = s.masked_fill(~causal, float("-inf"))
        outs.append(torch.softmax(s, dim=1) @ Vt[h // G])
    O = torch.stack(outs)
    ref_O, _ = fo.gated_attn(bits(Qb), bits(Kb), bits(Vb), g, lam, w)
    assert np.abs(O.detach().numpy() - ref_O).max() < 1e-12           # the same forward
    (O * torch.tensor(dO)).sum().backward()
    for got, want in ((dQ, Qt.grad), (dK, Kt.grad), (dV, Vt.grad), (dg, gt.grad)):
        assert np.abs(got - want.numpy()).max() < 1e-11
    # central differences of the oracle's forward with respect to a few assignment entries
    eps = 1e-6
    for a, b in ((0, 0), (n - 1, 1), (n // 2, 2)):
        gp = g.copy(); gp[a, b] += eps
        gm = g.copy(); gm[a, b] -= eps
        num = ((fo.gated_attn(bits(Qb), bits(Kb), bits(Vb), gp, lam, w)[0] - fo.gated_attn(bits(Qb), bits(Kb), bits(Vb), gm, lam, w)[0]) * dO).sum() / (2 * eps)
        assert abs(num - dg[a, b]) < 1e-6
    if w >= n:
        assert np.abs(dg).max() == 0.0


def test_gated_attention_backward_without_distant_pairs_has_no_assignment_gradient():
    rng = np.random.default_rng(2)
    import torch
    n, D = 5, 4
    bits = lambda x: torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    q, k, v = bits(rng.standard_normal((1, n, D))), bits(rng.standard_normal((1, n, D))), bits(rng.standard_normal((1, n, D)))
    g = rng.random((n, 2))
    dQ, dK, dV, dg = fo.gated_attn_backward(q, k, v, g, 5.0, n, rng.standard_normal((1, n, D)))
    assert np.abs(dg).max() == 0.0 and np.abs(dQ).max() > 0 and np.abs(dK).max() > 0 and np.abs(dV).max() > 0
