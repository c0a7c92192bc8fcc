"""FOCUS_LAYOUT_SORTED_LOCAL: the class-sorted pass over the pairs that share a group, the pass in token order over
the pairs kept by the window alone, and their logsumexp merge (paper Appendix D) -- against the fp64 oracle of the
whole rule, with the tolerances of the other layouts."""
import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2604_03260_b200 import binding as fb
from paper_2604_03260_b200 import inputs as fi
from tests.gpu_util import as_u32, assert_parity, compare_rows, gpu_assign, gpu_attn, gpu_tiles
from tests.test_gpu_attn import oracle_masks, run_case, to_dev
from tests.test_gpu_sorted import views
from tests.test_gpu_tiles import random_masks

pytestmark = pytest.mark.gpu
LAYOUT = fb.FOCUS_LAYOUT_SORTED_LOCAL


@pytest.mark.parametrize("n,w,K,t", [(300, 5, 4, 2), (4500, 300, 8, 2), (3000, 128, 6, 3), (2049, 5000, 4, 1)])
def test_ranges_list_only_the_sharing_classes(n, w, K, t):
    rng = np.random.default_rng(n + w)
    Hq, Hkv = 4, 2
    wl = fi.Workload("t", Hq, Hkv, 128, n, K, t, w)
    mq = random_masks(rng, Hq, n, K, t, False); mk = random_masks(rng, Hkv, n, K, t, False)
    ws, L = gpu_tiles(wl, to_dev(mq), to_dev(mk), LAYOUT)
    assert L.layout == LAYOUT and L.o_local > 0 and L.lse_local > L.o_local
    V = views(ws, L, Hq, Hkv)
    for h in range(Hq):
        hk = h // (Hq // Hkv)
        ref = fo.sorted_layout(mq[h], mk[hk], w)
        nk = len(ref["cls_k"])
        want = ref["ranges"].copy()
        for blk in range(want.shape[0]):
            jq = int(np.searchsorted(ref["seg_q"], blk * 256, side="right")) - 1      # class of the block
            for jk in range(nk):
                if (int(ref["cls_q"][jq]) & int(ref["cls_k"][jk])) == 0:
                    want[blk, jk] = 0
        got = V["qrange"][h, :want.shape[0], :nk]
        live = want[..., 1] > want[..., 0]
        assert np.array_equal(got[live], want[live])
        assert ((got[..., 1] - got[..., 0])[~live] <= 0).all()


@pytest.mark.parametrize("D", [64, 128, 256])
@pytest.mark.parametrize("n,w,K,t", [(1, 0, 4, 2), (130, 0, 4, 1), (300, 7, 4, 2), (777, 128, 8, 2), (1500, 127, 4, 1),
                                     (2048, 256, 4, 2), (2500, 5000, 4, 1), (1300, 300, 6, 3), (1024, 64, 1, 1), (5000, 200, 8, 2)])
def test_random_masks(D, n, w, K, t):
    wl = fi.Workload("o", 4, 2, D, n, K, t, w, seed=n + w + D)
    run_case(wl, layout=LAYOUT)


@pytest.mark.parametrize("D", [128, 256])
@pytest.mark.parametrize("w,K", [(0, 4), (100, 4), (300, 8)])
def test_run_structured_masks(w, K, D):
    wl = fi.Workload("b", 4, 2, D, 4000, K, 1, w, seed=w + K)
    rng = np.random.default_rng(w)
    masks = (random_masks(rng, 4, wl.n, K, 1, True), random_masks(rng, 2, wl.n, K, 1, True))
    run_case(wl, layout=LAYOUT, masks=masks)


def test_softcap_and_gqa():
    run_case(fi.Workload("c50", 8, 2, 128, 1500, 4, 1, 300, softcap=50.0, scale=1.0 / 16, seed=4), layout=LAYOUT)
    run_case(fi.Workload("c5", 4, 1, 256, 900, 4, 2, 50, softcap=5.0, scale=0.25, seed=3), layout=LAYOUT)


def test_rows_without_a_sharing_pair_come_from_the_window_pass_alone():
    """query masks and key masks disjoint: no pair shares a group, everything attended is window-only"""
    wl = fi.Workload("d", 4, 2, 128, 1200, 4, 1, 100, seed=9)
    mq = np.full((4, wl.n), 1, np.uint32); mk = np.full((2, wl.n), 2, np.uint32)
    run_case(wl, layout=LAYOUT, masks=(mq, mk))


def test_matches_the_class_sorted_layout_and_is_deterministic():
    wl = fi.Workload("eq", 8, 2, 128, 6000, 8, 2, 256, seed=21)
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    mq, mk = oracle_masks(wl, Q, K, C)
    dq, dk = to_dev(mq), to_dev(mk)
    ws1, _ = gpu_tiles(wl, dq, dk, 1)
    ws3, _ = gpu_tiles(wl, dq, dk, LAYOUT)
    O1, l1 = gpu_attn(wl, Q, K, V, dq, dk, ws1, 1)
    O3, l3 = gpu_attn(wl, Q, K, V, dq, dk, ws3, LAYOUT)
    O4, l4 = gpu_attn(wl, Q, K, V, dq, dk, ws3, LAYOUT)
    assert torch.equal(O3, O4) and torch.equal(l3, l4)
    assert (O1.float() - O3.float()).abs().max().item() <= 2e-2 and (l1 - l3).abs().max().item() <= 5e-3


def test_batch_of_two():
    wl = fi.Workload("bt", 4, 2, 128, 1700, 4, 2, 90, seed=5)
    shape = fb.make_shape(4, 2, wl.n, 128, 4, 2, 90, batch=2)
    g = torch.Generator(device="cuda"); g.manual_seed(3)
    Q = torch.randn((2, 4, wl.n, 128), generator=g, device="cuda").to(torch.bfloat16)
    K = torch.randn((2, 2, wl.n, 128), generator=g, device="cuda").to(torch.bfloat16)
    V = torch.randn((2, 2, wl.n, 128), generator=g, device="cuda").to(torch.bfloat16)
    rng = np.random.default_rng(1)
    mq = random_masks(rng, 8, wl.n, 4, 2, False); mk = random_masks(rng, 4, wl.n, 4, 2, False)
    ws = fb.alloc_workspace(shape, LAYOUT)
    fb.focus_build_tiles(shape, to_dev(mq), to_dev(mk), LAYOUT, ws)
    O = torch.full_like(Q, float("nan")); lse = torch.full((8, wl.n), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    fb.focus_attn_fwd(shape, Q, K, V, to_dev(mq), to_dev(mk), ws, LAYOUT, O, lse, status)
    torch.cuda.synchronize()
    assert status[0].item() == 0
    for b in range(2):
        stats = compare_rows(wl, Q[b], K[b], V[b], mq[4 * b:4 * b + 4], mk[2 * b:2 * b + 2], O[b], lse[4 * b:4 * b + 4])
        assert_parity(stats)


@pytest.mark.parametrize("name,per_head", [("cfg3", 48), ("cfg4", 32)])
def test_large_configs_sampled(name, per_head):
    wl = fi.WORKLOADS[name]
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    mq, _ = gpu_assign(wl, Q, C, wl.Hq)
    mk, _ = gpu_assign(wl, K, C, wl.Hkv)
    ws, _ = gpu_tiles(wl, mq, mk, LAYOUT)
    O, lse = gpu_attn(wl, Q, K, V, mq, mk, ws, LAYOUT)
    assert_parity(compare_rows(wl, Q, K, V, as_u32(mq), as_u32(mk), O, lse, rows=fi.sample_rows(wl, per_head)))
