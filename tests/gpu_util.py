"""Helpers for the GPU parity tests: run the CUDA path through the C-ABI binding, run the oracle on
the same bits, compare."""
import numpy as np
import torch

from oracle import focus_oracle as fo
from paper_2604_03260_b200 import binding as fb
from paper_2604_03260_b200 import inputs as fi

O_MAX_ABS = 2e-2      # bf16 inputs, fp32 accumulation, bf16 probabilities and outputs
O_MEAN_ABS = 2e-3
LSE_MAX_ABS = 5e-3


def gpu_assign(wl, X, C, H):
    shape = fb.shape_of(wl)
    masks = torch.empty((H, wl.n), dtype=torch.int32, device="cuda")
    near = torch.zeros(1, dtype=torch.int64, device="cuda")
    fb.focus_assign(shape, X, H, C, masks, near, 1e-5)
    torch.cuda.synchronize()
    count = int(near.item()) & (2 ** 64 - 1)
    assert count >> 63 == 0, "focus_assign set its fault flag (bit 63 of the near-tie word)"
    return masks, count


def gpu_tiles(wl, mq, mk, layout=0):
    shape = fb.shape_of(wl)
    ws = fb.alloc_workspace(shape, layout)
    fb.focus_build_tiles(shape, mq, mk, layout, ws)
    torch.cuda.synchronize()
    return ws, fb.focus_tiles_layout_of(shape, layout)


def gpu_attn(wl, Q, K, V, mq=None, mk=None, ws=None, layout=0):
    shape = fb.shape_of(wl)
    O = torch.full_like(Q, float("nan"))
    lse = torch.full((wl.Hq, wl.n), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    fb.focus_attn_fwd(shape, Q, K, V, mq, mk, ws, layout, O, lse, status)
    torch.cuda.synchronize()
    st = status.cpu().tolist()
    assert st[0] == 0, f"kernel reported an expired wait: {st}"
    return O, lse


def as_u32(t):
    return t.detach().cpu().numpy().view(np.uint32)


def masks_vs_oracle(wl, X, C, masks):
    """membership masks of the CUDA path against oracle.assign on the same bits: bit-exact except where the
    fp64 margin between the last group taken and the first one left is below 1e-5 (near-ties, counted).
    Returns (mismatches inside near-ties, near-ties)."""
    ref, margins = fo.assign(fi.bf16_bits(X), C.cpu().numpy(), wl.topk)
    got = as_u32(masks)
    bad = got != ref
    near = margins < 1e-5
    outside = bad & ~near
    assert not outside.any(), (f"{int(outside.sum())} masks differ from the oracle outside near-ties, first at "
                               f"(head, token) {np.argwhere(outside)[0].tolist()}")
    return int(bad.sum()), int(near.sum())


def compare_rows(wl, Q, K, V, mq_np, mk_np, O, lse, rows=None, dense=False):
    """oracle on the given rows (all rows when None) vs the GPU outputs; returns error statistics"""
    qb, kb, vb = fi.bf16_bits(Q), fi.bf16_bits(K), fi.bf16_bits(V)
    window = wl.n + 1 if dense else wl.window
    ref = fo.attn_rows(qb, kb, vb, mq_np, mk_np, window, scale=wl.logit_scale, softcap=wl.softcap, rows=rows)
    r = ref["rows"]
    Og = O.float().cpu().numpy().astype(np.float64)[r[:, 0], r[:, 1]]
    Lg = lse.cpu().numpy().astype(np.float64)[r[:, 0], r[:, 1]]
    assert np.isfinite(Og).all() and np.isfinite(Lg).all(), "non-finite GPU output"
    err = np.abs(Og - ref["O"])
    return dict(max_abs=float(err.max()), mean_abs=float(err.mean()), lse_max=float(np.abs(Lg - ref["lse"]).max()),
                rows=len(r), worst=r[int(err.max(axis=1).argmax())].tolist())


def assert_parity(stats):
    assert stats["max_abs"] <= O_MAX_ABS, stats
    assert stats["mean_abs"] <= O_MEAN_ABS, stats
    assert stats["lse_max"] <= LSE_MAX_ABS, stats
