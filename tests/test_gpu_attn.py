"""focus_attn_fwd vs the fp64 oracle, element by element, through the C ABI.
Tolerances (bf16 inputs, fp32 accumulation): O max-abs <= 2e-2, mean-abs <= 2e-3, lse max-abs <= 5e-3."""
import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2604_03260_b200 import binding as fb
from paper_2604_03260_b200 import inputs as fi
from tests.gpu_util import as_u32, assert_parity, compare_rows, gpu_assign, gpu_attn, gpu_tiles
from tests.test_gpu_tiles import random_masks

pytestmark = pytest.mark.gpu


def oracle_masks(wl, Q, K, C):
    mq, _ = fo.assign(fi.bf16_bits(Q), C.cpu().numpy(), wl.topk)
    mk, _ = fo.assign(fi.bf16_bits(K), C.cpu().numpy(), wl.topk)
    return mq, mk


def to_dev(m):
    return torch.from_numpy(m.view(np.int32)).cuda()


def run_case(wl, layout=0, masks=None, rows=None, dense=False):
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    if masks is None:
        mq, mk = oracle_masks(wl, Q, K, C)
    else:
        mq, mk = masks
    if dense:
        O, lse = gpu_attn(wl, Q, K, V)
    else:
        dq, dk = to_dev(mq), to_dev(mk)
        ws, _ = gpu_tiles(wl, dq, dk, layout)
        O, lse = gpu_attn(wl, Q, K, V, dq, dk, ws, layout)
    stats = compare_rows(wl, Q, K, V, mq, mk, O, lse, rows=rows, dense=dense)
    assert_parity(stats)
    return stats


@pytest.mark.parametrize("D", [64, 128, 256])
@pytest.mark.parametrize("n", [1, 100, 128, 129, 256, 257, 640, 1111])
def test_dense_causal_mode(D, n):
    wl = fi.Workload("d", 4, 2, D, n, 4, 2, 0, seed=n + D)
    run_case(wl, dense=True)


@pytest.mark.parametrize("D", [64, 128, 256])
@pytest.mark.parametrize("n,w,K,t", [(1, 0, 4, 2), (130, 0, 4, 1), (300, 7, 4, 2), (777, 128, 8, 2), (1000, 64, 4, 2),
                                     (1500, 127, 4, 1), (1500, 129, 2, 1), (2048, 256, 4, 2), (2500, 5000, 4, 1),
                                     (1300, 300, 32, 3), (1024, 64, 1, 1)])
def test_original_layout_random_masks(D, n, w, K, t):
    wl = fi.Workload("o", 4, 2, D, n, K, t, w, seed=n + w + D)
    run_case(wl)


@pytest.mark.parametrize("D", [128, 256])
@pytest.mark.parametrize("w,K", [(0, 4), (100, 4), (300, 8)])
def test_original_layout_skips_dead_tiles(w, K, D):
    """run-structured masks: whole far tiles die (skipped), others are full (mask-free)"""
    wl = fi.Workload("b", 4, 2, D, 4000, K, 1, w, seed=w + K)
    rng = np.random.default_rng(w)
    masks = (random_masks(rng, 4, wl.n, K, 1, True), random_masks(rng, 2, wl.n, K, 1, True))
    run_case(wl, masks=masks)


@pytest.mark.parametrize("D", [64, 128, 256])
def test_softcap(D):
    wl = fi.Workload("c", 4, 2, D, 900, 4, 2, 50, softcap=5.0, scale=0.25, seed=3)
    run_case(wl)
    run_case(wl, dense=True)
    wl = fi.Workload("c50", 4, 2, D, 1500, 4, 1, 300, softcap=50.0, scale=1.0 / 16, seed=4)
    run_case(wl)


def test_strided_tensors_and_determinism():
    wl = fi.Workload("st", 4, 2, 128, 700, 4, 2, 33, seed=12)
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    mq, mk = oracle_masks(wl, Q, K, C)
    dq, dk = to_dev(mq), to_dev(mk)
    ws, _ = gpu_tiles(wl, dq, dk, 0)
    O1, l1 = gpu_attn(wl, Q, K, V, dq, dk, ws, 0)
    O2, l2 = gpu_attn(wl, Q, K, V, dq, dk, ws, 0)
    assert torch.equal(O1, O2) and torch.equal(l1, l2)
    tr = lambda x: x.transpose(0, 1).contiguous().transpose(0, 1)       # [n, H, D] storage
    O3, l3 = gpu_attn(wl, tr(Q), tr(K), tr(V), dq, dk, ws, 0)
    assert torch.equal(O1, O3) and torch.equal(l1, l3)


def test_cfg1_all_rows_end_to_end():
    """assign -> build_tiles -> attn on the GPU; the oracle attends with the GPU's masks, and the
    masks themselves are compared (near-ties excepted) in test_gpu_assign"""
    wl = fi.WORKLOADS["cfg1"]
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    mq, _ = gpu_assign(wl, Q, C, wl.Hq)
    mk, _ = gpu_assign(wl, K, C, wl.Hkv)
    ws, _ = gpu_tiles(wl, mq, mk, 0)
    O, lse = gpu_attn(wl, Q, K, V, mq, mk, ws, 0)
    assert_parity(compare_rows(wl, Q, K, V, as_u32(mq), as_u32(mk), O, lse))
    Od, lsed = gpu_attn(wl, Q, K, V)
    assert_parity(compare_rows(wl, Q, K, V, as_u32(mq), as_u32(mk), Od, lsed, dense=True))


def test_cfg2_two_heads_all_rows_others_sampled():
    wl = fi.WORKLOADS["cfg2"]
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    mq, mk = oracle_masks(wl, Q, K, C)
    dq, dk = to_dev(mq), to_dev(mk)
    ws, _ = gpu_tiles(wl, dq, dk, 0)
    O, lse = gpu_attn(wl, Q, K, V, dq, dk, ws, 0)
    rows = [np.stack([np.full(wl.n, h), np.arange(wl.n)], 1) for h in (0, 31)]
    rows.append(fi.sample_rows(wl, 48))
    assert_parity(compare_rows(wl, Q, K, V, mq, mk, O, lse, rows=np.concatenate(rows)))


@pytest.mark.parametrize("D", [64, 128, 256])
@pytest.mark.parametrize("layout", [0, 1])
def test_peaked_logits_exercise_the_lazy_rescale(D, layout):
    """logit scale 8x the default: row maxima jump by far more than the rescale threshold between tiles, rows are
    nearly one-hot, masked tiles precede the first attended key of many rows.  An output row is then close to a
    single V row, values up to |4|, where the bf16 output grid alone is 2^-6 wide: the check is relative here,
    |err| <= 2^-7 |O| + 1e-2 (P and O each rounded to bf16), with lse to the usual absolute tolerance."""
    wl = fi.Workload("peak", 4, 2, D, 2300, 4, 1, 40, scale=8.0 / D ** 0.5, seed=90 + D)
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    mq, mk = oracle_masks(wl, Q, K, C)
    dq, dk = to_dev(mq), to_dev(mk)
    ws, _ = gpu_tiles(wl, dq, dk, layout)
    for dense in (False, True):
        O, lse = gpu_attn(wl, Q, K, V) if dense else gpu_attn(wl, Q, K, V, dq, dk, ws, layout)
        ref = fo.attn_rows(fi.bf16_bits(Q), fi.bf16_bits(K), fi.bf16_bits(V), mq, mk, wl.n + 1 if dense else wl.window,
                           scale=wl.logit_scale)
        og = O.float().cpu().numpy().reshape(-1, D).astype(np.float64)
        assert np.isfinite(og).all()
        err = np.abs(og - ref["O"])
        assert (err <= 2.0 ** -7 * np.abs(ref["O"]) + 1e-2).all(), float(err.max())
        assert err.mean() <= 2e-3
        assert np.abs(lse.cpu().numpy().reshape(-1) - ref["lse"]).max() <= 5e-3
