"""focus_assign vs the oracle: membership masks bit-exact except near-ties (margin < 1e-5), which
are counted and reported."""
import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2604_03260_b200 import inputs as fi
from tests.gpu_util import as_u32, gpu_assign

pytestmark = pytest.mark.gpu


def check(wl, X, C, H):
    masks, near_gpu = gpu_assign(wl, X, C, H)
    ref, margins = fo.assign(fi.bf16_bits(X), C.cpu().numpy(), wl.topk)
    got = as_u32(masks)
    bad = got != ref
    near = margins < 1e-5
    assert not (bad & ~near).any(), f"{int((bad & ~near).sum())} mismatches outside near-ties"
    # every mask has exactly topk bits inside the K groups
    pop = np.array([bin(int(x)).count("1") for x in np.unique(got)])
    assert (pop == wl.topk).all() and (np.unique(got) < (1 << wl.K)).all()
    # the GPU's own near-tie counter sees about the same set (fp32 vs fp64 margins)
    assert abs(near_gpu - int(near.sum())) <= max(8, int(0.5 * near.sum())), (near_gpu, int(near.sum()))
    return int(bad.sum()), int(near.sum())


@pytest.mark.parametrize("name", ["cfg1", "cfg2"])
def test_assign_configs(name):
    wl = fi.WORKLOADS[name]
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    check(wl, Q, C, wl.Hq)
    check(wl, K, C, wl.Hkv)


@pytest.mark.parametrize("D,K,t,n", [(64, 1, 1, 77), (64, 8, 3, 513), (128, 16, 4, 1000), (128, 32, 32, 300),
                                     (256, 4, 1, 1025), (256, 32, 5, 640), (128, 5, 2, 1)])
def test_assign_shapes(D, K, t, n):
    wl = fi.Workload("t", 4, 2, D, n, K, t, 8, seed=D + K + n)
    Q, Kt, V, C = fi.make_inputs(wl, "cuda")
    C = C * torch.linspace(0.5, 2.0, K, device="cuda")[None, :, None]      # non-unit centroids: still cosine
    check(wl, Q, C.contiguous(), wl.Hq)
    check(wl, Kt, C.contiguous(), wl.Hkv)


@pytest.mark.parametrize("Hq,Hkv,D,n,K,t", [(64, 16, 128, 2048 + 77, 4, 2), (32, 8, 256, 3000, 8, 2), (96, 48, 64, 1500, 16, 3)])
def test_assign_ranges_that_cross_heads(Hq, Hkv, D, n, K, t):
    """more tiles than resident blocks and few tiles per head: a block's range of tiles runs through several heads and
    KV heads, so it rebuilds its centroid operand on the way (at D = 256 with two pieces per tile)"""
    wl = fi.Workload("x", Hq, Hkv, D, n, K, t, 8, seed=Hq + D + n)
    Q, Kt, V, C = fi.make_inputs(wl, "cuda")
    check(wl, Q, C, wl.Hq)
    check(wl, Kt, C, wl.Hkv)


@pytest.mark.parametrize("name", ["cfg3", "cfg4", "M128k", "cfg5"])
def test_assign_large_configs_at_full_size(name):
    """every mask of the large configurations (clustered K = 8 at 32K, D = 256 top-1 at 64K, the 128K metric point,
    and 1M tokens, where element offsets pass 2^32) against the oracle; near-ties counted and reported"""
    wl = fi.WORKLOADS[name]
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    del V
    diff_k, near_k = check(wl, K, C, wl.Hkv)
    diff_q, near_q = check(wl, Q, C, wl.Hq)
    print(f"{wl.name}: near-ties Q {near_q} K {near_k} of {(wl.Hq + wl.Hkv) * wl.n} vectors; "
          f"masks differing inside near-ties Q {diff_q} K {diff_k}")
    assert near_q + near_k < 1e-3 * (wl.Hq + wl.Hkv) * wl.n + 16      # near-ties stay a rare event (measured: 2e-4 on cfg3)


def test_assign_clustered_and_ties():
    wl = fi.WORKLOADS["cfg3"].with_n(4096)
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    check(wl, Q, C, wl.Hq)
    # exact ties: duplicate centroids and zero vectors -> lowest indices win, on both sides
    wl2 = fi.Workload("ties", 2, 2, 64, 256, 4, 2, 8, seed=5)
    Q, K, V, C = fi.make_inputs(wl2, "cuda")
    C[:, 1] = C[:, 0]
    Q[:, ::7] = 0
    masks, _ = gpu_assign(wl2, Q, C.contiguous(), 2)
    ref, _ = fo.assign(fi.bf16_bits(Q), C.cpu().numpy(), 2)
    got = as_u32(masks)
    assert (got[:, ::7] == 0b11).all() and (ref[:, ::7] == 0b11).all()


def test_assign_strided_input():
    """[n, H, D] storage viewed as [H, n, D]"""
    wl = fi.Workload("s", 4, 2, 128, 600, 4, 2, 8, seed=9)
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    Qs = Q.transpose(0, 1).contiguous().transpose(0, 1)
    assert not Qs.is_contiguous()
    a, _ = gpu_assign(wl, Q, C, wl.Hq)
    b, _ = gpu_assign(wl, Qs, C, wl.Hq)
    assert torch.equal(a, b)
