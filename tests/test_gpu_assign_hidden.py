"""focus_assign_hidden (the paper's router: projected hidden state scored against centroids) vs the oracle:
masks bit-exact except near-ties, which are counted.  The margin is in score units; the near-tie threshold is
scaled to the size of the scores (fp32 accumulation over d_model terms, folded in a different order)."""
import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2604_03260_b200 import binding as fb
from paper_2604_03260_b200 import inputs as fi
from tests.gpu_util import as_u32

pytestmark = pytest.mark.gpu


def hidden_inputs(n, d, dg, K, seed, batch=1):
    g = torch.Generator(device="cuda"); g.manual_seed(seed)
    h = torch.randn((batch, n, d), generator=g, device="cuda").to(torch.bfloat16)
    Wg = torch.randn((d, dg), generator=g, device="cuda") / d ** 0.5
    C = torch.randn((K, dg), generator=g, device="cuda")
    bias = 0.3 * torch.randn(K, generator=g, device="cuda")
    return h, Wg, C, bias


@pytest.mark.parametrize("n,d,dg,K,t,use_bias,batch", [(1, 64, 16, 4, 2, False, 1), (300, 768, 16, 4, 2, True, 1),
                                                       (5000, 4096, 16, 8, 2, True, 1), (1000, 200, 7, 5, 1, False, 2),
                                                       (777, 1032, 32, 32, 3, True, 1), (129, 8, 4, 2, 2, False, 3),
                                                       # more tiles than resident blocks: a block's range runs from one sequence into the next
                                                       (8000, 520, 16, 4, 2, True, 8)])
def test_masks_match_the_oracle(n, d, dg, K, t, use_bias, batch):
    Hq, Hkv = 4, 2
    h, Wg, C, bias = hidden_inputs(n, d, dg, K, n + d, batch)
    shape = fb.make_shape(Hq, Hkv, n, 128, K, t, 16, batch=batch)
    folded = torch.empty((K, d), dtype=torch.float32, device="cuda")
    mq = torch.full((batch * Hq, n), -1, dtype=torch.int32, device="cuda")
    mk = torch.full((batch * Hkv, n), -1, dtype=torch.int32, device="cuda")
    near = torch.zeros(1, dtype=torch.int64, device="cuda")
    scale = float((h.float().norm(dim=-1).mean() * (Wg @ C.T).norm(dim=0).mean()).item())     # typical |score|
    eps = 2e-5 * scale
    fb.focus_assign_hidden(shape, h, Wg, C, bias if use_bias else None, folded, mq, mk, near, eps)
    torch.cuda.synchronize()
    assert torch.allclose(folded, (Wg @ C.T).T.contiguous(), rtol=1e-5, atol=1e-6)
    got_q, got_k = as_u32(mq).reshape(batch, Hq, n), as_u32(mk).reshape(batch, Hkv, n)
    total_near = 0
    for b in range(batch):
        ref, margins = fo.assign_hidden(fi.bf16_bits(h[b]), Wg.cpu().numpy(), C.cpu().numpy(), t,
                                        bias.cpu().numpy() if use_bias else None)
        near_ref = margins < eps
        total_near += int(near_ref.sum())
        for hh in range(Hq):
            assert not ((got_q[b, hh] != ref) & ~near_ref).any()
        for hh in range(Hkv):
            assert np.array_equal(got_k[b, hh], got_q[b, 0])        # one mask per token, shared by every head and role
        pop = np.array([bin(int(x)).count("1") for x in np.unique(got_q[b])])
        assert (pop == t).all()
    assert abs(int(near.item()) - total_near) <= max(8, total_near)


def test_feeds_the_attention_path():
    """router masks -> build_tiles (class-sorted) -> attention, against the oracle attending with the same masks"""
    from tests.gpu_util import assert_parity, compare_rows, gpu_attn, gpu_tiles
    wl = fi.Workload("r", 4, 2, 128, 1500, 4, 1, 64, seed=31)
    Q, K, V, _ = fi.make_inputs(wl, "cuda")
    h, Wg, C, bias = hidden_inputs(wl.n, 512, 16, wl.K, 77)
    shape = fb.shape_of(wl)
    folded = torch.empty((wl.K, 512), dtype=torch.float32, device="cuda")
    mq = torch.empty((wl.Hq, wl.n), dtype=torch.int32, device="cuda"); mk = torch.empty((wl.Hkv, wl.n), dtype=torch.int32, device="cuda")
    fb.focus_assign_hidden(shape, h, Wg, C, bias, folded, mq, mk)
    for layout in (0, 1):
        ws, _ = gpu_tiles(wl, mq, mk, layout)
        O, lse = gpu_attn(wl, Q, K, V, mq, mk, ws, layout)
        assert_parity(compare_rows(wl, Q, K, V, as_u32(mq), as_u32(mk), O, lse))
