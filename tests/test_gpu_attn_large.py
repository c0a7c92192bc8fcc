"""The large parity configurations, in the launch configuration bench.py times, checked on sampled
query rows (seeded draws plus boundary rows per head) that the oracle computes one by one."""
import numpy as np
import pytest
import torch

from paper_2604_03260_b200 import binding as fb
from paper_2604_03260_b200 import inputs as fi
from tests.gpu_util import as_u32, assert_parity, compare_rows, gpu_assign, gpu_attn, gpu_tiles, masks_vs_oracle

pytestmark = pytest.mark.gpu


def run_sampled(name, per_head, layout=0, dense_too=False):
    wl = fi.WORKLOADS[name]
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    mq, _ = gpu_assign(wl, Q, C, wl.Hq)
    mk, _ = gpu_assign(wl, K, C, wl.Hkv)
    # the masks both sides use below are the oracle's own except at counted near-ties
    masks_vs_oracle(wl, Q, C, mq)
    masks_vs_oracle(wl, K, C, mk)
    ws, L = gpu_tiles(wl, mq, mk, layout)
    O, lse = gpu_attn(wl, Q, K, V, mq, mk, ws, layout)
    rows = fi.sample_rows(wl, per_head)
    stats = compare_rows(wl, Q, K, V, as_u32(mq), as_u32(mk), O, lse, rows=rows)
    assert_parity(stats)
    # properties that hold at any size: every output row was written and is finite
    assert torch.isfinite(lse).all() and torch.isfinite(O.float()).all()
    # kept-pair fraction sanity against the exact counter
    cnt = torch.zeros(wl.Hq, dtype=torch.int64, device="cuda")
    fb.focus_count_kept(fb.shape_of(wl), mq, ws, cnt)
    torch.cuda.synchronize()
    frac = cnt.sum().item() / wl.dense_pairs()
    if dense_too:
        del O, lse
        O, lse = gpu_attn(wl, Q, K, V)
        assert_parity(compare_rows(wl, Q, K, V, as_u32(mq), as_u32(mk), O, lse, rows=rows[::4], dense=True))
    return stats, frac


@pytest.mark.parametrize("name,per_head,lo,hi", [("cfg3", 48, 0.3, 0.9), ("cfg4", 48, 0.30, 0.40), ("M128k", 64, 0.82, 0.86),
                                                 ("cfg5", 256, 0.82, 0.85)])
def test_class_sorted_layout_on_the_large_configs(name, per_head, lo, hi):
    stats, frac = run_sampled(name, per_head, layout=1)
    assert lo < frac < hi


def test_cfg3_clustered_skewed_groups():
    stats, frac = run_sampled("cfg3", 64, dense_too=True)
    assert 0.3 < frac < 0.9


def test_cfg4_head_dim_256_softcap():
    stats, frac = run_sampled("cfg4", 64, dense_too=True)
    assert 0.30 < frac < 0.40          # 1/4 of far pairs + the window


def test_metric_point_128k():
    stats, frac = run_sampled("M128k", 96)
    assert 0.82 < frac < 0.86


def test_cfg5_one_million_tokens():
    stats, frac = run_sampled("cfg5", 256)
    assert 0.82 < frac < 0.85


@pytest.mark.parametrize("name,lo,hi", [("Mruns", 0.80, 0.90), ("Mruns1", 0.22, 0.32)])
def test_run_structured_memberships_at_the_metric_shape(name, lo, hi):
    """memberships coherent over positions: in the original layout whole far tiles die (skipped) and others are
    attended without any mask; sampled rows against the oracle, tile counters against what the draw implies"""
    stats, frac = run_sampled(name, 64)
    assert lo < frac < hi
    wl = fi.WORKLOADS[name]
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    mq, _ = gpu_assign(wl, Q, C, wl.Hq)
    mk, _ = gpu_assign(wl, K, C, wl.Hkv)
    ws, L = gpu_tiles(wl, mq, mk, 0)
    far, live, full = fb.ws_view(ws, L.counters, 8, torch.int64)[:3].tolist()
    assert 0 < full < live < far
    assert live < (0.95 if wl.topk == 2 else 0.6) * far          # a good part of the far tiles is never visited
    assert full > 0.2 * live                                      # and a good part of the rest needs no mask
