"""focus_build_tiles / focus_count_kept vs the oracle's tile reference and exact pair count."""
import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2604_03260_b200 import binding as fb
from paper_2604_03260_b200 import inputs as fi
from tests.gpu_util import gpu_tiles

pytestmark = pytest.mark.gpu


def random_masks(rng, H, n, K, t, blocky):
    m = np.zeros((H, n), np.uint32)
    for h in range(H):
        if blocky:      # long runs of one group, so that tiles really die / become full
            g = (np.arange(n) // rng.integers(100, 400) + h) % K
            m[h] = 1 << g
            flip = rng.random(n) < 0.002
            m[h][flip] = 1 << rng.integers(0, K, flip.sum())
        else:
            for i in range(n):
                m[h, i] = sum(1 << int(g) for g in rng.choice(K, size=t, replace=False))
    return m


@pytest.mark.parametrize("n,w,K,t,blocky", [(1, 0, 1, 1, False), (127, 5, 4, 2, False), (1000, 64, 4, 2, True),
                                            (4500, 300, 8, 2, True), (4500, 0, 4, 1, True), (2049, 5000, 4, 1, True),
                                            (5000, 128, 32, 3, False)])
def test_summaries_live_set_and_counts(n, w, K, t, blocky):
    rng = np.random.default_rng(n + w)
    Hq, Hkv = 4, 2
    wl = fi.Workload("t", Hq, Hkv, 128, n, K, t, w)
    mq = random_masks(rng, Hq, n, K, t, blocky); mk = random_masks(rng, Hkv, n, K, t, blocky)
    dq = torch.from_numpy(mq.view(np.int32)).cuda(); dk = torch.from_numpy(mk.view(np.int32)).cuda()
    ws, L = gpu_tiles(wl, dq, dk, 0)
    ref = fo.tile_reference(mq, mk, w, 128, 128)

    def view(off, count, dt=torch.int32):
        return fb.ws_view(ws, off, count, dt).cpu().numpy()

    assert np.array_equal(view(L.orq, Hq * L.nqt).view(np.uint32).reshape(Hq, L.nqt), ref["orq"])
    assert np.array_equal(view(L.andq, Hq * L.nqt).view(np.uint32).reshape(Hq, L.nqt), ref["andq"])
    assert np.array_equal(view(L.ork, Hkv * L.nkt).view(np.uint32).reshape(Hkv, L.nkt), ref["ork"])
    assert np.array_equal(view(L.andk, Hkv * L.nkt).view(np.uint32).reshape(Hkv, L.nkt), ref["andk"])
    # group column bitmaps: bit j of tile b, group g <-> key 128 b + j is a member of g
    gb = view(L.gbits, Hkv * L.nkt * K * 4).view(np.uint32).reshape(Hkv, L.nkt, K, 4)
    bits = ((gb[..., None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(Hkv, L.nkt, K, 128)
    member = np.zeros((Hkv, L.nkt * 128, K), np.uint32)
    member[:, :n] = (mk[..., None] >> np.arange(K, dtype=np.uint32)) & 1
    assert np.array_equal(bits, member.reshape(Hkv, L.nkt, 128, K).transpose(0, 1, 3, 2))
    # live bitmap, per-row counts, totals
    lv = view(L.live, Hq * L.nqt * L.nkw).view(np.uint32).reshape(Hq, L.nqt, L.nkw)
    live = ((lv[..., None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(Hq, L.nqt, L.nkw * 32)[..., :L.nkt].astype(bool)
    assert np.array_equal(live, ref["live"])
    assert np.array_equal(view(L.live_cnt, Hq * L.nqt).reshape(Hq, L.nqt), ref["live"].sum(-1))
    counters = view(L.counters, 8, torch.int64)
    assert counters[0] == ref["far"].sum() * Hq and counters[1] == ref["live"].sum() and counters[2] == ref["full"].sum()
    if blocky and n >= 1000 and w < n:
        assert 0 < counters[1] < counters[0]          # some far tiles die, some live
    # exact attended-pair count
    cnt = torch.zeros(Hq, dtype=torch.int64, device="cuda")
    fb.focus_count_kept(fb.shape_of(wl), dq, ws, cnt)
    torch.cuda.synchronize()
    assert cnt.cpu().tolist() == fo.kept_pairs(mq, mk, w).tolist()


def test_count_kept_on_cfg2_masks():
    wl = fi.WORKLOADS["cfg2"]
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    shape = fb.shape_of(wl)
    mq = torch.empty((wl.Hq, wl.n), dtype=torch.int32, device="cuda")
    mk = torch.empty((wl.Hkv, wl.n), dtype=torch.int32, device="cuda")
    fb.focus_assign(shape, Q, wl.Hq, C, mq)
    fb.focus_assign(shape, K, wl.Hkv, C, mk)
    ws, L = gpu_tiles(wl, mq, mk, 0)
    cnt = torch.zeros(wl.Hq, dtype=torch.int64, device="cuda")
    fb.focus_count_kept(shape, mq, ws, cnt)
    torch.cuda.synchronize()
    ref = fo.kept_pairs(mq.cpu().numpy().view(np.uint32), mk.cpu().numpy().view(np.uint32), wl.window)
    assert cnt.cpu().tolist() == ref.tolist()
    frac = cnt.sum().item() / wl.dense_pairs()
    assert 0.80 < frac < 0.90          # 5/6 of far pairs + the window (0.854 for uniform memberships)
