"""tcgen05 / TMA building blocks in isolation: one S = A B^T tile and one O = P V tile."""
import pytest
import torch

from paper_2604_03260_b200 import binding as fb

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("D", [64, 128, 256])
def test_umma_tiles_match_matmul(D):
    g = torch.Generator(device="cuda").manual_seed(D)
    a = torch.randn(128, D, generator=g, device="cuda").bfloat16()
    b = torch.randn(128, D, generator=g, device="cuda").bfloat16()
    p = torch.rand(128, 128, generator=g, device="cuda").bfloat16()
    v = torch.randn(128, D, generator=g, device="cuda").bfloat16()
    s = torch.zeros(128, 128, device="cuda")
    o = torch.zeros(128, D, device="cuda")
    st = torch.zeros(4, dtype=torch.int32, device="cuda")
    fb.focus_selftest_umma(D, a, b, p, v, s, o, st)
    torch.cuda.synchronize()
    assert st[0].item() == 0
    s_ref = a.double() @ b.double().T
    o_ref = p.double() @ v.double()
    assert (s.double() - s_ref).abs().max().item() < 1e-3 * max(1.0, s_ref.abs().max().item())
    assert (o.double() - o_ref).abs().max().item() < 1e-3 * max(1.0, o_ref.abs().max().item())


def test_umma_tiles_shared_by_a_cta_pair_match_matmul():
    g = torch.Generator(device="cuda").manual_seed(2)
    a = torch.randn(256, 128, generator=g, device="cuda").bfloat16()
    b = torch.randn(128, 128, generator=g, device="cuda").bfloat16()
    p = torch.rand(256, 128, generator=g, device="cuda").bfloat16()
    v = torch.randn(128, 128, generator=g, device="cuda").bfloat16()
    s = torch.zeros(256, 128, device="cuda")
    o = torch.zeros(256, 128, device="cuda")
    st = torch.zeros(4, dtype=torch.int32, device="cuda")
    fb.focus_selftest_umma_pair(a, b, p, v, s, o, st)
    torch.cuda.synchronize()
    assert st[0].item() == 0
    s_ref = a.double() @ b.double().T
    o_ref = p.double() @ v.double()
    assert (s.double() - s_ref).abs().max().item() < 1e-3 * max(1.0, s_ref.abs().max().item())
    assert (o.double() - o_ref).abs().max().item() < 1e-3 * max(1.0, o_ref.abs().max().item())
