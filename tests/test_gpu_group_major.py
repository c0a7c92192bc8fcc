"""FOCUS_LAYOUT_GROUP_MAJOR: queries sorted by class, keys laid out as K lists (a key once per group it belongs to), a
sharing pair attended under its lowest shared group, window-only pairs from the pass in token order, merged through
the logsumexps (paper Sec. 2 "Sort tokens by group"; Sec. 3.6 top-k membership; Appendix D "Disjoint decomposition"
and "Merge").  The structures against the oracle's definition, the attention against the fp64 oracle of the rule."""
import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2604_03260_b200 import binding as fb
from paper_2604_03260_b200 import inputs as fi
from tests.gpu_util import as_u32, assert_parity, compare_rows, gpu_assign, gpu_attn, gpu_tiles, masks_vs_oracle
from tests.test_gpu_attn import oracle_masks, run_case, to_dev
from tests.test_gpu_sorted import INT_MAX, MAXC, views
from tests.test_gpu_tiles import random_masks

pytestmark = pytest.mark.gpu
LAYOUT = fb.FOCUS_LAYOUT_GROUP_MAJOR


@pytest.mark.parametrize("n,w,K,t,blocky", [(1, 0, 1, 1, False), (300, 5, 4, 2, False), (1000, 64, 4, 2, True),
                                            (4500, 300, 8, 2, False), (4500, 0, 4, 1, True), (3000, 128, 6, 3, False),
                                            (2100, 50, 11, 2, False), (1500, 10, 32, 1, False)])
def test_structures_match_their_definition(n, w, K, t, blocky):
    rng = np.random.default_rng(n + w + 2)
    Hq, Hkv = 4, 2
    wl = fi.Workload("t", Hq, Hkv, 128, n, K, t, w)
    mq = random_masks(rng, Hq, n, K, t, blocky); mk = random_masks(rng, Hkv, n, K, t, blocky)
    ws, L = gpu_tiles(wl, to_dev(mq), to_dev(mk), LAYOUT)
    assert L.layout == LAYOUT and L.gbits_s > 0 and L.nkp >= n * t
    V = views(ws, L, Hq, Hkv)
    gb = fb.ws_view(ws, L.gbits_s, Hkv * (L.nkp // 128) * K * 4, torch.int32).cpu().numpy().view(np.uint32)
    gb = gb.reshape(Hkv, L.nkp // 128, K, 4)
    assert V["counters"][4] == 0
    for h in range(Hq):
        hk = h // (Hq // Hkv)
        ref = fo.group_major_layout(mq[h], mk[hk], K)
        nq = len(ref["cls_q"])
        assert V["ncls_q"][h] == nq and V["ncls_k"][hk] == K
        assert np.array_equal(V["cls_q"][h, :nq], ref["cls_q"])
        assert np.array_equal(V["cls_k"][hk, :K], 1 << np.arange(K, dtype=np.uint32)) and (V["cls_k"][hk, K:] == 0).all()
        assert np.array_equal(V["cnt_k"][hk, :K], ref["cnt_k"]) and np.array_equal(V["seg_k"][hk, :K + 1], ref["seg_k"])
        used_q, used_k = int(ref["seg_q"][-1]), int(ref["seg_k"][-1])
        assert V["seg_k"][hk, MAXC] == used_k
        assert np.array_equal(V["perm_q"][h, :used_q], ref["perm_q"])
        assert np.array_equal(V["perm_k"][hk, :used_k], ref["perm_k"]) and (V["perm_k"][hk, used_k:] == INT_MAX).all()
        nblk = used_q // 256
        assert np.array_equal(V["qrange"][h, :nblk, :K], ref["ranges"])
        assert (V["qrange"][h, nblk:] == 0).all() and (V["qrange"][h, :, K:] == 0).all()
        ntile = used_k // 128
        bits = ((gb[hk, :ntile, :, :, None] >> np.arange(32, dtype=np.uint32)) & 1).astype(bool).reshape(ntile, K, 128)
        assert np.array_equal(bits, ref["gbits"])


@pytest.mark.parametrize("D", [64, 128, 256])
@pytest.mark.parametrize("n,w,K,t", [(1, 0, 4, 2), (130, 0, 4, 1), (300, 7, 4, 2), (777, 128, 8, 2), (1500, 127, 4, 1),
                                     (2048, 256, 4, 2), (2500, 5000, 4, 1), (1300, 300, 6, 3), (1024, 64, 1, 1), (5000, 200, 8, 2),
                                     (3000, 100, 4, 4), (2200, 64, 11, 2)])
def test_random_masks(D, n, w, K, t):
    wl = fi.Workload("o", 4, 2, D, n, K, t, w, seed=n + w + D)
    run_case(wl, layout=LAYOUT)


@pytest.mark.parametrize("D", [128, 256])
@pytest.mark.parametrize("w,K,t", [(0, 4, 1), (100, 4, 2), (300, 8, 2)])
def test_run_structured_masks(w, K, t, D):
    wl = fi.Workload("b", 4, 2, D, 4000, K, t, w, seed=w + K)
    rng = np.random.default_rng(w)
    masks = (random_masks(rng, 4, wl.n, K, t, True), random_masks(rng, 2, wl.n, K, t, True))
    run_case(wl, layout=LAYOUT, masks=masks)


def test_softcap_gqa_and_peaked_logits():
    run_case(fi.Workload("c50", 8, 2, 128, 1500, 4, 2, 300, softcap=50.0, scale=1.0 / 16, seed=4), layout=LAYOUT)
    run_case(fi.Workload("c5", 4, 1, 256, 900, 4, 2, 50, softcap=5.0, scale=0.25, seed=3), layout=LAYOUT)


def test_more_classes_than_the_class_sorted_layouts_hold_on_the_key_side():
    """K = 16, top-2 on the key side gives up to 120 key classes: refused by the class-sorted layouts, fine here as long
    as the query side stays within the class table (queries use 2 of the first 8 groups: 28 classes)"""
    wl = fi.Workload("many", 4, 2, 128, 3000, 16, 2, 40, seed=8)
    rng = np.random.default_rng(3)
    pick = lambda rows, groups: np.array([[sum(1 << int(g) for g in rng.choice(groups, 2, replace=False)) for _ in range(wl.n)]
                                          for _ in range(rows)], np.uint32)
    run_case(wl, layout=LAYOUT, masks=(pick(4, 8), pick(2, 16)))


def test_matches_the_split_class_sorted_layout_and_is_deterministic():
    wl = fi.Workload("eq", 8, 2, 128, 6000, 8, 2, 256, seed=21)
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    mq, mk = oracle_masks(wl, Q, K, C)
    dq, dk = to_dev(mq), to_dev(mk)
    ws3, _ = gpu_tiles(wl, dq, dk, fb.FOCUS_LAYOUT_SORTED_LOCAL)
    ws4, _ = gpu_tiles(wl, dq, dk, LAYOUT)
    O3, l3 = gpu_attn(wl, Q, K, V, dq, dk, ws3, fb.FOCUS_LAYOUT_SORTED_LOCAL)
    O4, l4 = gpu_attn(wl, Q, K, V, dq, dk, ws4, LAYOUT)
    O4b, l4b = gpu_attn(wl, Q, K, V, dq, dk, ws4, LAYOUT)
    assert torch.equal(O4, O4b) and torch.equal(l4, l4b)
    assert (O3.float() - O4.float()).abs().max().item() <= 2e-2 and (l3 - l4).abs().max().item() <= 5e-3


def test_cfg3_at_full_size():
    wl = fi.WORKLOADS["cfg3"]
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    mq, _ = gpu_assign(wl, Q, C, wl.Hq)
    mk, _ = gpu_assign(wl, K, C, wl.Hkv)
    masks_vs_oracle(wl, Q, C, mq)
    masks_vs_oracle(wl, K, C, mk)
    ws, L = gpu_tiles(wl, mq, mk, LAYOUT)
    O, lse = gpu_attn(wl, Q, K, V, mq, mk, ws, LAYOUT)
    assert torch.isfinite(lse).all() and torch.isfinite(O.float()).all()
    assert_parity(compare_rows(wl, Q, K, V, as_u32(mq), as_u32(mk), O, lse, rows=fi.sample_rows(wl, 64)))
