"""batch > 1: every entry point indexes heads batch-major (b * H + h); each batch element must equal the
single-sequence result of the oracle on that element's tensors and masks."""
import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2604_03260_b200 import binding as fb
from paper_2604_03260_b200 import inputs as fi
from tests.gpu_util import LSE_MAX_ABS, O_MAX_ABS, O_MEAN_ABS, as_u32

pytestmark = pytest.mark.gpu


def batched_inputs(wl, B):
    parts = [fi.make_inputs(fi.Workload(wl.name, wl.Hq, wl.Hkv, wl.D, wl.n, wl.K, wl.topk, wl.window, seed=wl.seed + 17 * b), "cuda")
             for b in range(B)]
    Q = torch.stack([p[0] for p in parts]); K = torch.stack([p[1] for p in parts]); V = torch.stack([p[2] for p in parts])
    return Q, K, V, parts[0][3]            # one centroid set for the whole batch (it is indexed by KV head only)


@pytest.mark.parametrize("D,layout", [(64, 0), (128, 0), (128, 1), (256, 1)])
def test_hot_path_with_a_batch(D, layout):
    B = 3
    wl = fi.Workload("b", 4, 2, D, 1100, 4, 2, 48, seed=40 + D)
    shape = fb.make_shape(wl.Hq, wl.Hkv, wl.n, wl.D, wl.K, wl.topk, wl.window, batch=B)
    Q, K, V, C = batched_inputs(wl, B)
    mq = torch.empty((B * wl.Hq, wl.n), dtype=torch.int32, device="cuda")
    mk = torch.empty((B * wl.Hkv, wl.n), dtype=torch.int32, device="cuda")
    fb.focus_assign(shape, Q, wl.Hq, C, mq)
    fb.focus_assign(shape, K, wl.Hkv, C, mk)
    ws = fb.alloc_workspace(shape, layout)
    fb.focus_build_tiles(shape, mq, mk, layout, ws)
    O = torch.full_like(Q, float("nan"))
    lse = torch.full((B * wl.Hq, wl.n), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    fb.focus_attn_fwd(shape, Q, K, V, mq, mk, ws, layout, O, lse, status)
    cnt = torch.zeros(B * wl.Hq, dtype=torch.int64, device="cuda")
    fb.focus_count_kept(shape, mq, ws, cnt)
    torch.cuda.synchronize()
    assert status[0].item() == 0
    mqn, mkn = as_u32(mq).reshape(B, wl.Hq, wl.n), as_u32(mk).reshape(B, wl.Hkv, wl.n)
    lse_b = lse.reshape(B, wl.Hq, wl.n)
    for b in range(B):
        ref_m, margins = fo.assign(fi.bf16_bits(Q[b]), C.cpu().numpy(), wl.topk)
        assert not ((mqn[b] != ref_m) & ~(margins < 1e-5)).any()
        ref = fo.attn_rows(fi.bf16_bits(Q[b]), fi.bf16_bits(K[b]), fi.bf16_bits(V[b]), mqn[b], mkn[b], wl.window)
        err = np.abs(O[b].float().cpu().numpy().reshape(-1, wl.D).astype(np.float64) - ref["O"])
        lerr = np.abs(lse_b[b].cpu().numpy().reshape(-1).astype(np.float64) - ref["lse"])
        assert err.max() <= O_MAX_ABS and err.mean() <= O_MEAN_ABS and lerr.max() <= LSE_MAX_ABS
        assert cnt.reshape(B, wl.Hq)[b].cpu().tolist() == fo.kept_pairs(mqn[b], mkn[b], wl.window).tolist()


def test_decode_with_a_batch():
    B = 2
    wl = fi.Workload("bd", 8, 2, 128, 3000, 4, 1, 100, seed=77)
    shape = fb.make_shape(wl.Hq, wl.Hkv, wl.n, wl.D, wl.K, wl.topk, wl.window, batch=B)
    Q, K, V, C = batched_inputs(wl, B)
    mq = torch.empty((B * wl.Hq, wl.n), dtype=torch.int32, device="cuda")
    mk = torch.empty((B * wl.Hkv, wl.n), dtype=torch.int32, device="cuda")
    fb.focus_assign(shape, Q, wl.Hq, C, mq)
    fb.focus_assign(shape, K, wl.Hkv, C, mk)
    q_new = Q[:, :, -1, :].contiguous()                    # [B, Hq, D]
    mq_new = mq[:, -1].contiguous()                        # [B * Hq]
    o = torch.full((B, wl.Hq, wl.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B * wl.Hq,), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(fb.focus_decode_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    fb.focus_decode_step(shape, q_new, K, V, mq_new, mk, o, lse, ws)
    torch.cuda.synchronize()
    mqn, mkn = as_u32(mq).reshape(B, wl.Hq, wl.n), as_u32(mk).reshape(B, wl.Hkv, wl.n)
    rows = np.stack([np.arange(wl.Hq), np.full(wl.Hq, wl.n - 1)], 1)
    for b in range(B):
        ref = fo.attn_rows(fi.bf16_bits(Q[b]), fi.bf16_bits(K[b]), fi.bf16_bits(V[b]), mqn[b], mkn[b], wl.window, rows=rows)
        err = np.abs(o[b].float().cpu().numpy().astype(np.float64) - ref["O"])
        lerr = np.abs(lse.reshape(B, wl.Hq)[b].cpu().numpy().astype(np.float64) - ref["lse"])
        assert err.max() <= O_MAX_ABS and err.mean() <= O_MEAN_ABS and lerr.max() <= LSE_MAX_ABS
