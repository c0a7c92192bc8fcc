"""tcgen05 / TMA building blocks in isolation: one S = A B^T tile and one O = P V tile."""
import pytest
import torch

from paper_2604_03260_b200 import binding as fb
from paper_2604_03260_b200 import inputs as fi

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


@pytest.mark.parametrize("D", [64, 128, 256])
def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(D):
    """one stage of the K/V ring is never filled: the waiting role gives up after its limit, the kernel says where,
    releases tensor memory and returns; the next ordinary launch in the same process is correct"""
    from tests.gpu_util import assert_parity, compare_rows, gpu_attn
    import numpy as np
    wl = fi.Workload("stall", 2, 1, D, 1500, 4, 2, 8, seed=40 + D)
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    shape = fb.shape_of(wl)
    O = torch.zeros_like(Q)
    lse = torch.zeros((wl.Hq, wl.n), dtype=torch.float32, device="cuda")
    st = torch.zeros(4, dtype=torch.int32, device="cuda")
    fb.focus_selftest_stalled_wait(shape, Q, K, V, O, lse, 2_000_000, st)
    torch.cuda.synchronize()                       # returns: nothing hangs, nothing faults
    code = st.cpu().tolist()
    # whichever role started waiting first reports: the MMA role for the stage itself (21-23), the producer for the ring
    # slot that is never handed back (10, 11), or a softmax role for the S / O that never comes (30, 31, 40, 41)
    assert code[0] == 1 and code[1] in (10, 11, 21, 22, 23, 30, 31, 40, 41), code
    assert 0 <= code[3] < 148
    masks = np.full((wl.Hq, wl.n), 0b11, np.uint32), np.full((wl.Hkv, wl.n), 0b11, np.uint32)
    O2, lse2 = gpu_attn(wl, Q, K, V)                # asserts a clean status itself
    assert_parity(compare_rows(wl, Q, K, V, masks[0], masks[1], O2, lse2, dense=True))


@pytest.mark.parametrize("pair,N,ts,pattern", [(0, 128, 0, 0), (0, 128, 1, 0), (0, 256, 0, 0), (1, 128, 0, 0), (1, 128, 1, 0),
                                               (0, 128, 0, 1), (0, 128, 0, 3), (1, 128, 0, 3), (0, 64, 0, 2), (0, 96, 0, 3)])
def test_mma_rate_probe_runs_and_reports_a_plausible_rate(pair, N, ts, pattern):
    """the probe's waits end, and the rate it reports lies between a tenth of and a little above the nominal one"""
    rounds = 500
    res = torch.full((3,), -1, dtype=torch.int64, device="cuda")
    fb.focus_selftest_mma_rate(pair, N, ts, pattern, rounds, res)
    torch.cuda.synchronize()
    cycles, ns, fault = (int(x) for x in res.tolist())
    assert fault == 0 and cycles > 0 and ns > 0
    chains = 1 if pattern == 0 else 2
    rate = chains * 2.0 * 128 * N * 128 * rounds / cycles
    assert 0.1 * 8192 < rate < 1.05 * 8192, rate


def test_mma_rate_probe_refuses_shapes_without_room_in_tensor_memory():
    res = torch.zeros(3, dtype=torch.int64, device="cuda")
    for args in ((0, 256, 1, 0), (0, 256, 0, 1), (1, 64, 0, 0), (0, 128, 1, 2), (0, 100, 0, 0)):
        with pytest.raises(fb.FocusError):
            fb.focus_selftest_mma_rate(*args, 100, res)
