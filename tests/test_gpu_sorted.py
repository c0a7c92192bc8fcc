"""Class-sorted layout: focus_build_tiles(layout 1) against the oracle's sorted-layout reference, and
focus_attn_fwd in that layout against the fp64 oracle (same tolerances as the original layout)."""
import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2604_03260_b200 import binding as fb
from paper_2604_03260_b200 import inputs as fi
from tests.gpu_util import as_u32, assert_parity, compare_rows, gpu_assign, gpu_attn, gpu_tiles
from tests.test_gpu_attn import oracle_masks, run_case, to_dev
from tests.test_gpu_tiles import random_masks

pytestmark = pytest.mark.gpu
MAXC = fb.FOCUS_MAX_CLASSES
INT_MAX = np.iinfo(np.int32).max


def views(ws, L, Hq, Hkv):
    v = lambda off, count: fb.ws_view(ws, off, count, torch.int32).cpu().numpy()
    nqblk = L.nqp // 256
    return dict(
        ncls_q=v(L.ncls_q, Hq), ncls_k=v(L.ncls_k, Hkv),
        cls_q=v(L.cls_q, Hq * MAXC).view(np.uint32).reshape(Hq, MAXC), cls_k=v(L.cls_k, Hkv * MAXC).view(np.uint32).reshape(Hkv, MAXC),
        cnt_q=v(L.cnt_q, Hq * MAXC).reshape(Hq, MAXC), cnt_k=v(L.cnt_k, Hkv * MAXC).reshape(Hkv, MAXC),
        seg_q=v(L.seg_q, Hq * (MAXC + 1)).reshape(Hq, MAXC + 1), seg_k=v(L.seg_k, Hkv * (MAXC + 1)).reshape(Hkv, MAXC + 1),
        perm_q=v(L.perm_q, Hq * L.nqp).reshape(Hq, L.nqp), perm_k=v(L.perm_k, Hkv * L.nkp).reshape(Hkv, L.nkp),
        qrange=v(L.qrange, Hq * nqblk * MAXC * 2).reshape(Hq, nqblk, MAXC, 2),
        order=v(L.order, Hq * nqblk * 2).reshape(Hkv, (Hq // Hkv) * nqblk, 2),
        counters=fb.ws_view(ws, L.counters, 8, torch.int64).cpu().numpy())


@pytest.mark.parametrize("n,w,K,t,blocky", [(1, 0, 1, 1, False), (300, 5, 4, 2, False), (1000, 64, 4, 2, True),
                                            (4500, 300, 8, 2, False), (4500, 0, 4, 1, True), (2049, 5000, 4, 1, False),
                                            (3000, 128, 6, 3, False)])
def test_sorted_structures(n, w, K, t, blocky):
    rng = np.random.default_rng(n + w + 1)
    Hq, Hkv = 4, 2
    wl = fi.Workload("t", Hq, Hkv, 128, n, K, t, w)
    mq = random_masks(rng, Hq, n, K, t, blocky); mk = random_masks(rng, Hkv, n, K, t, blocky)
    ws, L = gpu_tiles(wl, to_dev(mq), to_dev(mk), 1)
    V = views(ws, L, Hq, Hkv)
    assert V["counters"][4] == 0
    total_tiles = 0
    for h in range(Hq):
        hk = h // (Hq // Hkv)
        ref = fo.sorted_layout(mq[h], mk[hk], w)
        nq, nk = len(ref["cls_q"]), len(ref["cls_k"])
        assert V["ncls_q"][h] == nq and V["ncls_k"][hk] == nk
        assert np.array_equal(V["cls_q"][h, :nq], ref["cls_q"]) and np.array_equal(V["cls_k"][hk, :nk], ref["cls_k"])
        assert np.array_equal(V["cnt_q"][h, :nq], ref["cnt_q"]) and np.array_equal(V["cnt_k"][hk, :nk], ref["cnt_k"])
        assert np.array_equal(V["seg_q"][h, :nq + 1], ref["seg_q"]) and np.array_equal(V["seg_k"][hk, :nk + 1], ref["seg_k"])
        used_q, used_k = int(ref["seg_q"][-1]), int(ref["seg_k"][-1])
        assert V["seg_q"][h, MAXC] == used_q and V["seg_k"][hk, MAXC] == used_k
        assert np.array_equal(V["perm_q"][h, :used_q], ref["perm_q"]) and (V["perm_q"][h, used_q:] == -1).all()
        assert np.array_equal(V["perm_k"][hk, :used_k], ref["perm_k"]) and (V["perm_k"][hk, used_k:] == INT_MAX).all()
        nblk = used_q // 256
        assert np.array_equal(V["qrange"][h, :nblk, :nk], ref["ranges"])
        assert (V["qrange"][h, nblk:] == 0).all() and (V["qrange"][h, :, nk:] == 0).all()
        total_tiles += int((ref["ranges"][..., 1] - ref["ranges"][..., 0]).sum())
    assert V["counters"][3] == total_tiles
    # block order: every (head, block) of a KV head group exactly once, costs non-increasing up to the bucket width
    cost = (V["qrange"][..., 1] - V["qrange"][..., 0]).sum(-1)
    G = Hq // Hkv
    for hk in range(Hkv):
        pairs = V["order"][hk]
        assert sorted(map(tuple, pairs.tolist())) == [(hk * G + g, b) for g in range(G) for b in range(L.nqp // 256)]
        c = cost[pairs[:, 0], pairs[:, 1]]
        slack = max(1, (L.nkp // 128 + 2046) // 2047)
        assert (c[1:] <= c[:-1] + slack).all()


def test_too_many_mask_values_is_refused():
    wl = fi.Workload("x", 2, 1, 128, 600, 32, 3, 10)
    shape = fb.shape_of(wl)
    ws = fb.alloc_workspace(shape, 1)
    m = torch.zeros((2, 600), dtype=torch.int32, device="cuda")
    with pytest.raises(fb.FocusError) as e:
        fb.focus_build_tiles(shape, m, m[:1], 1, ws)
    assert e.value.status == -2
    # arbitrary masks with more than 64 distinct values under a small C(K, topk): caught on the device
    wl = fi.Workload("y", 2, 1, 128, 600, 7, 3, 10)
    shape = fb.shape_of(wl)
    ws = fb.alloc_workspace(shape, 1)
    mq = torch.arange(600, dtype=torch.int32, device="cuda").remainder(100).add(1).repeat(2, 1).contiguous()
    mk = mq[:1].contiguous()
    fb.focus_build_tiles(shape, mq, mk, 1, ws)
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    O = torch.zeros_like(Q); lse = torch.zeros((2, 600), dtype=torch.float32, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    fb.focus_attn_fwd(shape, Q, K, V, mq, mk, ws, 1, O, lse, status)
    torch.cuda.synchronize()
    assert status[0].item() == 2


@pytest.mark.parametrize("D", [64, 128, 256])
@pytest.mark.parametrize("n,w,K,t", [(1, 0, 4, 2), (130, 0, 4, 1), (300, 7, 4, 2), (777, 128, 8, 2), (1000, 64, 4, 2),
                                     (1500, 127, 4, 1), (1500, 129, 2, 1), (2048, 256, 4, 2), (2500, 5000, 4, 1),
                                     (1300, 300, 6, 3), (1024, 64, 1, 1), (5000, 200, 4, 2)])
def test_sorted_layout_random_masks(D, n, w, K, t):
    wl = fi.Workload("o", 4, 2, D, n, K, t, w, seed=n + w + D)
    run_case(wl, layout=1)


@pytest.mark.parametrize("D", [128, 256])
@pytest.mark.parametrize("w,K", [(0, 4), (100, 4), (300, 8)])
def test_sorted_layout_run_structured_masks(w, K, D):
    wl = fi.Workload("b", 4, 2, D, 4000, K, 1, w, seed=w + K)
    rng = np.random.default_rng(w)
    masks = (random_masks(rng, 4, wl.n, K, 1, True), random_masks(rng, 2, wl.n, K, 1, True))
    run_case(wl, layout=1, masks=masks)


@pytest.mark.parametrize("D", [64, 128, 256])
def test_sorted_layout_softcap(D):
    wl = fi.Workload("c", 4, 2, D, 900, 4, 2, 50, softcap=5.0, scale=0.25, seed=3)
    run_case(wl, layout=1)
    wl = fi.Workload("c50", 4, 2, D, 1500, 4, 1, 300, softcap=50.0, scale=1.0 / 16, seed=4)
    run_case(wl, layout=1)


def test_sorted_equals_original_layout_and_is_deterministic():
    wl = fi.Workload("eq", 8, 2, 128, 3000, 4, 2, 100, seed=21)
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    mq, mk = oracle_masks(wl, Q, K, C)
    dq, dk = to_dev(mq), to_dev(mk)
    ws0, _ = gpu_tiles(wl, dq, dk, 0)
    ws1, _ = gpu_tiles(wl, dq, dk, 1)
    O0, l0 = gpu_attn(wl, Q, K, V, dq, dk, ws0, 0)
    O1, l1 = gpu_attn(wl, Q, K, V, dq, dk, ws1, 1)
    O2, l2 = gpu_attn(wl, Q, K, V, dq, dk, ws1, 1)
    assert torch.equal(O1, O2) and torch.equal(l1, l2)
    assert (O0.float() - O1.float()).abs().max().item() <= 2e-2 and (l0 - l1).abs().max().item() <= 5e-3
    # the kept-pair counter reads the same summaries in both workspaces
    c0 = torch.zeros(wl.Hq, dtype=torch.int64, device="cuda"); c1 = torch.zeros_like(c0)
    fb.focus_count_kept(fb.shape_of(wl), dq, ws0, c0); fb.focus_count_kept(fb.shape_of(wl), dq, ws1, c1)
    torch.cuda.synchronize()
    assert torch.equal(c0, c1) and c0.cpu().tolist() == fo.kept_pairs(mq, mk, wl.window).tolist()


def test_cfg1_all_rows_sorted_end_to_end():
    wl = fi.WORKLOADS["cfg1"]
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    mq, _ = gpu_assign(wl, Q, C, wl.Hq)
    mk, _ = gpu_assign(wl, K, C, wl.Hkv)
    ws, _ = gpu_tiles(wl, mq, mk, 1)
    O, lse = gpu_attn(wl, Q, K, V, mq, mk, ws, 1)
    assert_parity(compare_rows(wl, Q, K, V, as_u32(mq), as_u32(mk), O, lse))


def test_cfg2_sorted_two_heads_all_rows_others_sampled():
    wl = fi.WORKLOADS["cfg2"]
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    mq, mk = oracle_masks(wl, Q, K, C)
    dq, dk = to_dev(mq), to_dev(mk)
    ws, _ = gpu_tiles(wl, dq, dk, 1)
    O, lse = gpu_attn(wl, Q, K, V, dq, dk, ws, 1)
    rows = [np.stack([np.full(wl.n, h), np.arange(wl.n)], 1) for h in (3, 28)]
    rows.append(fi.sample_rows(wl, 48))
    assert_parity(compare_rows(wl, Q, K, V, mq, mk, O, lse, rows=np.concatenate(rows)))


def test_auto_layout_runs_whichever_it_picks():
    for wl, expect in ((fi.Workload("a0", 4, 2, 128, 3000, 4, 1, 64, seed=51), 0),
                       (fi.Workload("a1", 4, 2, 128, 17000, 4, 1, 64, seed=52), 1),
                       (fi.Workload("a3", 4, 2, 128, 17000, 8, 1, 512, seed=53), 3)):
        assert fb.focus_tiles_layout_of(fb.shape_of(wl), fb.FOCUS_LAYOUT_AUTO).layout == expect
        run_case(wl, layout=fb.FOCUS_LAYOUT_AUTO, rows=fi.sample_rows(wl, 200))
