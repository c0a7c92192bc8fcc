"""focus_decode_step (one new query against the cached keys and values) vs the fp64 oracle's row n-1 of the
forward definition.  bf16 operands, fp32 accumulation, probabilities rounded to bf16 before P V: O max-abs <= 2e-2,
mean-abs <= 2e-3, lse max-abs <= 5e-3 -- the tolerances of the forward pass."""
import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2604_03260_b200 import binding as fb
from paper_2604_03260_b200 import inputs as fi
from tests.gpu_util import LSE_MAX_ABS, O_MAX_ABS, O_MEAN_ABS

pytestmark = pytest.mark.gpu


def run_decode(wl, seed_masks=0, structured=False):
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    rng = np.random.default_rng(wl.n + seed_masks)
    def draw(H):
        m = np.zeros((H, wl.n), np.uint32)
        for h in range(H):
            if structured:
                m[h] = np.uint32(1) << ((np.arange(wl.n) // 300 + h) % wl.K).astype(np.uint32)
            else:
                picks = np.argsort(rng.random((wl.n, wl.K)), axis=1)[:, :wl.topk]
                for r in range(wl.topk):
                    m[h] |= np.uint32(1) << picks[:, r].astype(np.uint32)
        return m
    mq, mk = draw(wl.Hq), draw(wl.Hkv)
    shape = fb.shape_of(wl)
    q_new = Q[:, wl.n - 1, :].contiguous()                       # [Hq, D]
    mq_new = torch.from_numpy(mq[:, wl.n - 1].copy().view(np.int32)).cuda()
    dk = torch.from_numpy(mk.view(np.int32)).cuda()
    o = torch.full((wl.Hq, wl.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((wl.Hq,), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(fb.focus_decode_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    fb.focus_decode_step(shape, q_new, K, V, mq_new, dk, o, lse, ws)
    torch.cuda.synchronize()
    rows = np.stack([np.arange(wl.Hq), np.full(wl.Hq, wl.n - 1)], 1)
    ref = fo.attn_rows(fi.bf16_bits(Q), fi.bf16_bits(K), fi.bf16_bits(V), mq, mk, wl.window, scale=wl.logit_scale,
                       softcap=wl.softcap, rows=rows)
    og = o.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(og).all()
    err = np.abs(og - ref["O"])
    lerr = np.abs(lse.cpu().numpy().astype(np.float64) - ref["lse"])
    assert err.max() <= O_MAX_ABS and err.mean() <= O_MEAN_ABS and lerr.max() <= LSE_MAX_ABS, (err.max(), err.mean(), lerr.max())
    return ref["kept"]


@pytest.mark.parametrize("D", [64, 128, 256])
@pytest.mark.parametrize("Hq,Hkv,n,w,K,t", [(4, 2, 1, 0, 4, 2), (4, 4, 127, 0, 4, 1), (8, 2, 129, 5, 4, 2), (4, 2, 1000, 64, 4, 2),
                                            (16, 2, 3000, 0, 8, 2), (4, 2, 5000, 6000, 4, 1), (6, 3, 20000, 512, 4, 1),
                                            (2, 2, 777, 100, 1, 1)])
def test_decode_matches_oracle_row(D, Hq, Hkv, n, w, K, t):
    run_decode(fi.Workload("d", Hq, Hkv, D, n, K, t, w, seed=n + D))


def test_decode_structured_masks_and_softcap():
    kept = run_decode(fi.Workload("s", 4, 2, 128, 9000, 4, 1, 100, seed=5), structured=True)
    assert kept.max() < 9000 * 0.5                 # whole chunks of keys are skipped (not even copied)
    run_decode(fi.Workload("c", 4, 2, 256, 4000, 4, 1, 300, softcap=50.0, scale=1.0 / 16, seed=6))
    run_decode(fi.Workload("c5", 4, 2, 64, 2000, 4, 2, 30, softcap=5.0, scale=0.25, seed=7))


def test_decode_argument_checks():
    wl = fi.Workload("a", 18, 2, 128, 100, 4, 2, 8)
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    shape = fb.shape_of(wl)
    ws = torch.empty(max(16, fb.focus_decode_workspace_bytes(shape)), dtype=torch.uint8, device="cuda")
    o = torch.empty((18, 128), dtype=torch.bfloat16, device="cuda"); lse = torch.empty(18, device="cuda")
    m = torch.zeros((18, 100), dtype=torch.int32, device="cuda")
    with pytest.raises(fb.FocusError) as e:        # 9 query heads per KV head
        fb.focus_decode_step(shape, Q[:, -1].contiguous(), K, V, m[:, 0].contiguous(), m[:2], o, lse, ws)
    assert e.value.status == -2
    wl = fi.Workload("a", 4, 2, 128, 100, 4, 2, 8)
    shape = fb.shape_of(wl)
    with pytest.raises(fb.FocusError) as e:        # workspace too small
        fb.focus_decode_step(shape, Q[:4, -1].contiguous(), K, V, m[:4, 0].contiguous(), m[:2], o[:4], lse[:4], ws[:16])
    assert e.value.status == -3
