"""Training-time forward (paper Sec. 2: Eq. 1 with Sinkhorn normalisation, Eq. 2 soft gate) vs the oracle:
router scores, Sinkhorn assignments, and the gated attention forward over all causal pairs."""
import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2604_03260_b200 import binding as fb
from paper_2604_03260_b200 import inputs as fi
from tests.gpu_util import LSE_MAX_ABS, O_MAX_ABS, O_MEAN_ABS

pytestmark = pytest.mark.gpu


def padded(x, ld):
    """[.., K] -> [.., ld] with zeros"""
    out = torch.zeros(x.shape[:-1] + (ld,), dtype=torch.float32, device=x.device)
    out[..., :x.shape[-1]] = x
    return out.contiguous()


@pytest.mark.parametrize("n,d,dg,K,batch", [(1, 64, 16, 4, 1), (300, 768, 16, 4, 1), (5000, 4096, 16, 8, 1), (1000, 200, 7, 5, 2),
                                            (777, 1032, 32, 32, 1), (129, 8, 4, 12, 3)])
def test_router_scores(n, d, dg, K, batch):
    g = torch.Generator(device="cuda"); g.manual_seed(n + d)
    h = torch.randn((batch, n, d), generator=g, device="cuda").to(torch.bfloat16)
    Wg = torch.randn((d, dg), generator=g, device="cuda") / d ** 0.5
    C = torch.randn((K, dg), generator=g, device="cuda")
    ld = fb.focus_soft_ld(K)
    assert ld >= K and ld in (4, 8, 16, 32)
    shape = fb.make_shape(4, 2, n, 128, K, 1, 16, batch=batch)
    folded = torch.empty((K, d), dtype=torch.float32, device="cuda")
    S = torch.full((batch, n, ld), float("nan"), dtype=torch.float32, device="cuda")
    fb.focus_router_scores(shape, h, Wg, C, folded, S)
    torch.cuda.synchronize()
    got = S.cpu().numpy().astype(np.float64)
    assert (got[..., K:] == 0).all()
    for b in range(batch):
        ref = fo.router_scores(fi.bf16_bits(h[b]), Wg.cpu().numpy(), C.cpu().numpy())
        # fp32 accumulation over d terms, folded in a different order
        assert np.abs(got[b, :, :K] - ref).max() <= 2e-5 * max(1.0, np.abs(ref).max()) * max(1.0, d / 512) ** 0.5


@pytest.mark.parametrize("n,K,tau,iters,batch,spread", [(1, 4, 0.1, 10, 1, 0.3), (300, 4, 0.5, 10, 1, 1.0), (5000, 8, 0.1, 10, 1, 0.3),
                                                        (70000, 8, 0.1, 10, 1, 0.3), (777, 32, 0.1, 3, 2, 0.5), (513, 1, 0.1, 2, 1, 1.0),
                                                        (1000, 5, 0.1, 1, 3, 0.3), (4096, 8, 0.1, 10, 1, 10.0), (400000, 4, 0.1, 10, 1, 0.3)])
def test_sinkhorn(n, K, tau, iters, batch, spread):
    g = torch.Generator(device="cuda"); g.manual_seed(n * 7 + K)
    ld = fb.focus_soft_ld(K)
    S = padded(spread * torch.randn((batch, n, K), generator=g, device="cuda"), ld)
    shape = fb.make_shape(4, 2, n, 128, K, 1, 16, batch=batch)
    ws = torch.empty(fb.focus_sinkhorn_workspace_bytes(shape, iters), dtype=torch.uint8, device="cuda")
    out = torch.full_like(S, float("nan"))
    fb.focus_sinkhorn(shape, S, tau, iters, ws, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy().astype(np.float64)
    assert (got[..., K:] == 0).all()
    Sh = S.cpu().numpy().astype(np.float64)
    for b in range(batch):
        ref = fo.sinkhorn(Sh[b, :, :K], tau, iters)
        np.testing.assert_allclose(got[b, :, :K], ref, rtol=5e-4, atol=1e-7)
        np.testing.assert_allclose(got[b, :, :K].sum(axis=1), 1.0, atol=1e-5)
    # in place
    fb.focus_sinkhorn(shape, S, tau, iters, ws, S)
    torch.cuda.synchronize()
    assert torch.equal(S, out)


def gate_case(Hq, Hkv, n, D, K, seed, batch=1):
    g = torch.Generator(device="cuda"); g.manual_seed(seed)
    Q = torch.randn((batch, Hq, n, D), generator=g, device="cuda").to(torch.bfloat16)
    Kt = torch.randn((batch, Hkv, n, D), generator=g, device="cuda").to(torch.bfloat16)
    V = torch.randn((batch, Hkv, n, D), generator=g, device="cuda").to(torch.bfloat16)
    scores = 0.3 * torch.randn((batch, n, K), generator=g, device="cuda")
    soft = np.stack([fo.sinkhorn(scores[b].cpu().numpy().astype(np.float64), 0.1, 10) for b in range(batch)])
    gt = padded(torch.from_numpy(soft).float().cuda(), fb.focus_soft_ld(K))
    return Q, Kt, V, gt


def run_gate(Q, Kt, V, gt, K, w, lam):
    batch, Hq, n, D = Q.shape
    shape = fb.make_shape(Hq, Kt.shape[1], n, D, K, 1, w, batch=batch)
    O = torch.full_like(Q, float("nan"))
    lse = torch.full((batch * Hq, n), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    fb.focus_gate_attn_fwd(shape, Q, Kt, V, gt, lam, O, lse, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0
    return O, lse.reshape(batch, Hq, n)


def check_gate(Q, Kt, V, gt, K, w, lam, O, lse, rows=None):
    for b in range(Q.shape[0]):
        refO, refL = fo.gated_attn(fi.bf16_bits(Q[b]), fi.bf16_bits(Kt[b]), fi.bf16_bits(V[b]),
                                   gt[b, :, :K].cpu().numpy().astype(np.float64), lam, w, None, rows)
        r = np.arange(Q.shape[2]) if rows is None else np.asarray(rows)
        Og = O[b].float().cpu().numpy().astype(np.float64)[:, r]
        Lg = lse[b].cpu().numpy().astype(np.float64)[:, r]
        assert np.isfinite(Og).all() and np.isfinite(Lg).all()
        err = np.abs(Og - refO)
        assert err.max() <= O_MAX_ABS and err.mean() <= O_MEAN_ABS, (err.max(), err.mean())
        assert np.abs(Lg - refL).max() <= LSE_MAX_ABS, np.abs(Lg - refL).max()


@pytest.mark.parametrize("Hq,Hkv,n,D,K,w,lam,batch", [(2, 2, 1, 64, 4, 0, 5.0, 1), (4, 2, 700, 64, 4, 64, 8.0, 1), (4, 2, 1000, 128, 4, 0, 5.0, 1),
                                                      (4, 1, 1500, 128, 8, 300, 20.0, 1), (2, 1, 900, 256, 8, 100, 10.0, 1),
                                                      (2, 2, 640, 128, 5, 2000, 10.0, 1), (2, 1, 517, 128, 2, 33, 6.0, 2),
                                                      (2, 2, 384, 256, 4, 0, 30.0, 2),
                                                      # assignment rows of 16 and 32 floats (K up to 32, the paper's widest ablation)
                                                      (2, 1, 700, 128, 12, 64, 10.0, 1), (2, 2, 900, 128, 16, 0, 8.0, 1),
                                                      (4, 2, 1100, 128, 32, 200, 10.0, 1), (2, 1, 520, 64, 32, 50, 12.0, 2),
                                                      (2, 1, 600, 64, 9, 0, 5.0, 1), (2, 1, 777, 256, 16, 100, 10.0, 1),
                                                      (2, 2, 300, 256, 11, 0, 20.0, 1), (2, 1, 1, 128, 32, 0, 5.0, 1)])
def test_gated_attention_all_rows(Hq, Hkv, n, D, K, w, lam, batch):
    Q, Kt, V, gt = gate_case(Hq, Hkv, n, D, K, 100 + n, batch)
    O, lse = run_gate(Q, Kt, V, gt, K, w, lam)
    check_gate(Q, Kt, V, gt, K, w, lam, O, lse)


def test_gate_changes_the_result():
    """the gated output differs from plain causal attention by far more than the tolerance (the gate is live)"""
    Q, Kt, V, gt = gate_case(2, 2, 1024, 128, 4, 9)
    O, _ = run_gate(Q, Kt, V, gt, 4, 16, 10.0)
    O2, _ = run_gate(Q, Kt, V, gt, 4, 5000, 10.0)
    assert (O.float() - O2.float()).abs().max().item() > 0.2


def test_gated_attention_refuses_what_it_has_no_room_for():
    """D = 256 with more than 16 groups: the gate buffers would leave no room for the K/V ring"""
    Q, Kt, V, gt = gate_case(2, 1, 256, 256, 32, 9)
    shape = fb.make_shape(2, 1, 256, 256, 32, 1, 16)
    O = torch.empty_like(Q); lse = torch.empty((2, 256), dtype=torch.float32, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(fb.FocusError, match="K <= 16 at D = 256"):
        fb.focus_gate_attn_fwd(shape, Q, Kt, V, gt, 5.0, O, lse, status)


def test_gated_attention_32_groups_sampled_rows():
    """K = 32 at a length with several items per CTA (three-stage K/V ring beside the gate buffers)"""
    n, K, w, lam = 20000, 32, 1024, 10.0
    Q, Kt, V, gt = gate_case(4, 2, n, 128, K, 57)
    O, lse = run_gate(Q, Kt, V, gt, K, w, lam)
    rng = np.random.default_rng(6)
    rows = np.unique(np.concatenate([rng.integers(0, n, 12), [0, w, w + 1, n - 1]]))
    check_gate(Q, Kt, V, gt, K, w, lam, O, lse, rows)


@pytest.mark.parametrize("D,n", [(128, 40000), (256, 20000)])
def test_gated_attention_sampled_rows(D, n):
    """several items per CTA and a ragged last tile; rows sampled, plus the rows around the window edge"""
    K, w, lam = 8, 2048, 10.0
    Q, Kt, V, gt = gate_case(4, 2, n, D, K, 55)
    O, lse = run_gate(Q, Kt, V, gt, K, w, lam)
    rng = np.random.default_rng(3)
    rows = np.unique(np.concatenate([rng.integers(0, n, 40), [0, 1, w - 1, w, w + 1, 127, 128, n // 2, n - 128, n - 1]]))
    check_gate(Q, Kt, V, gt, K, w, lam, O, lse, rows)


def test_refusals():
    Q, Kt, V, gt = gate_case(2, 2, 256, 128, 4, 1)
    O = torch.empty_like(Q); lse = torch.empty((2, 256), dtype=torch.float32, device="cuda")
    with pytest.raises(fb.FocusError):      # softcap
        fb.focus_gate_attn_fwd(fb.make_shape(2, 2, 256, 128, 4, 1, 16, softcap=30.0), Q, Kt, V, gt, 5.0, O, lse)
    shape = fb.make_shape(2, 2, 256, 128, 4, 1, 16)
    small = torch.empty(8, dtype=torch.uint8, device="cuda")
    with pytest.raises(fb.FocusError):      # workspace too small
        fb.focus_sinkhorn(shape, gt, 0.1, 10, small, gt)
    ws = torch.empty(fb.focus_sinkhorn_workspace_bytes(shape, 10), dtype=torch.uint8, device="cuda")
    with pytest.raises(fb.FocusError):      # temperature
        fb.focus_sinkhorn(shape, gt, 0.0, 10, ws, gt)


def test_chain_hidden_to_gated_output():
    """hidden states -> scores -> Sinkhorn -> gated attention, every step on the GPU; the oracle runs the same chain"""
    n, d, dg, K, D, w, lam = 1200, 512, 16, 8, 128, 128, 10.0
    g = torch.Generator(device="cuda"); g.manual_seed(77)
    h = torch.randn((1, n, d), generator=g, device="cuda").to(torch.bfloat16)
    Wg = torch.randn((d, dg), generator=g, device="cuda") / d ** 0.5
    C = 0.2 * torch.randn((K, dg), generator=g, device="cuda")
    Q, Kt, V, _ = gate_case(4, 2, n, D, K, 78)
    shape = fb.make_shape(4, 2, n, D, K, 1, w)
    folded = torch.empty((K, d), dtype=torch.float32, device="cuda")
    S = torch.empty((1, n, fb.focus_soft_ld(K)), dtype=torch.float32, device="cuda")
    fb.focus_router_scores(shape, h, Wg, C, folded, S)
    ws = torch.empty(fb.focus_sinkhorn_workspace_bytes(shape, 10), dtype=torch.uint8, device="cuda")
    fb.focus_sinkhorn(shape, S, 0.1, 10, ws, S)
    O, lse = run_gate(Q, Kt, V, S, K, w, lam)
    ref_g = fo.sinkhorn(fo.router_scores(fi.bf16_bits(h[0]), Wg.cpu().numpy(), C.cpu().numpy()), 0.1, 10)
    np.testing.assert_allclose(S[0, :, :K].cpu().numpy(), ref_g, rtol=2e-3, atol=1e-6)
    refO, refL = fo.gated_attn(fi.bf16_bits(Q[0]), fi.bf16_bits(Kt[0]), fi.bf16_bits(V[0]), ref_g, lam, w)
    err = np.abs(O[0].float().cpu().numpy() - refO)
    assert err.max() <= O_MAX_ABS and err.mean() <= O_MEAN_ABS
    assert np.abs(lse[0].cpu().numpy() - refL).max() <= LSE_MAX_ABS


def test_gated_attention_at_the_metric_point_shape():
    """32 / 8 heads, D = 128, 131072 tokens, K = 4, w = 2048 (the launch the bench times): sampled rows of every head"""
    n, K, w, lam = 131072, 4, 2048, 10.0
    Q, Kt, V, gt = gate_case(32, 8, n, 128, K, 61)
    O, lse = run_gate(Q, Kt, V, gt, K, w, lam)
    rng = np.random.default_rng(4)
    rows = np.unique(np.concatenate([rng.integers(0, n, 6), [0, w, w + 1, n // 2, n - 1]]))
    check_gate(Q, Kt, V, gt, K, w, lam, O, lse, rows)


@pytest.mark.parametrize("n,K,tau,iters,batch,spread", [(1, 4, 0.1, 10, 1, 0.3), (300, 4, 0.5, 10, 1, 1.0), (5000, 8, 0.1, 10, 1, 0.3),
                                                        (70000, 8, 0.1, 10, 1, 0.3), (777, 32, 0.1, 3, 2, 0.5), (513, 1, 0.1, 2, 1, 1.0),
                                                        (1000, 5, 0.1, 1, 3, 0.3), (4096, 8, 0.1, 10, 1, 10.0), (2000, 12, 0.2, 6, 1, 0.5)])
def test_sinkhorn_backward(n, K, tau, iters, batch, spread):
    """d loss / d scores through the Sinkhorn steps against the oracle's tape-based derivative (fp64); the oracle's
    derivative is pinned on the CPU by central differences of its own forward"""
    g = torch.Generator(device="cuda"); g.manual_seed(n * 11 + K)
    ld = fb.focus_soft_ld(K)
    S = padded(spread * torch.randn((batch, n, K), generator=g, device="cuda"), ld)
    dG = padded(torch.randn((batch, n, K), generator=g, device="cuda"), ld)
    dG[..., K:] = 7.0                                    # entries beyond K are ignored
    shape = fb.make_shape(4, 2, n, 128, K, 1, 16, batch=batch)
    ws = torch.empty(fb.focus_sinkhorn_bwd_workspace_bytes(shape, iters), dtype=torch.uint8, device="cuda")
    dS = torch.full_like(S, float("nan"))
    fb.focus_sinkhorn_bwd(shape, S, tau, iters, ws, dG, dS)
    torch.cuda.synchronize()
    got = dS.cpu().numpy().astype(np.float64)
    assert (got[..., K:] == 0).all()
    Sh, dGh = S.cpu().numpy().astype(np.float64), dG.cpu().numpy().astype(np.float64)
    for b in range(batch):
        ref = fo.sinkhorn_backward(Sh[b, :, :K], tau, iters, dGh[b, :, :K])
        scale = max(np.abs(ref).max(), 1e-30)
        err = np.abs(got[b, :, :K] - ref).max() / scale
        # fp32 rows (exp, a K-term dot product with cancellation) against fp64; column sums are fp64 on both sides
        assert err <= 2e-4, (err, scale)
    # in place over dg, and twice in a row into the same workspace
    fb.focus_sinkhorn_bwd(shape, S, tau, iters, ws, dG, dG)
    torch.cuda.synchronize()
    assert torch.equal(dG, dS)


def test_sinkhorn_backward_is_orthogonal_to_what_sinkhorn_ignores():
    """adding a constant to a column of the scores scales that column of exp(S / tau), which the first column division
    undoes: the assignments do not change, so the derivative sums to zero over every column"""
    n, K, tau, iters = 3000, 8, 0.1, 10
    g = torch.Generator(device="cuda"); g.manual_seed(3)
    S = 0.5 * torch.randn((1, n, 8), generator=g, device="cuda")
    dG = torch.randn((1, n, 8), generator=g, device="cuda")
    shape = fb.make_shape(4, 2, n, 128, K, 1, 16)
    ws = torch.empty(fb.focus_sinkhorn_bwd_workspace_bytes(shape, iters), dtype=torch.uint8, device="cuda")
    dS = torch.empty_like(S)
    fb.focus_sinkhorn_bwd(shape, S, tau, iters, ws, dG, dS)
    d = dS[0].double()
    size = d.abs().max().item()
    assert d.sum(dim=0).abs().max().item() <= 1e-3 * size * n ** 0.5


def test_sinkhorn_one_million_tokens():
    n, K, tau, iters = 1 << 20, 8, 0.1, 10
    g = torch.Generator(device="cuda"); g.manual_seed(8)
    S = padded(0.3 * torch.randn((1, n, K), generator=g, device="cuda"), 8)
    shape = fb.make_shape(32, 8, n, 128, K, 1, 2048)
    ws = torch.empty(fb.focus_sinkhorn_workspace_bytes(shape, iters), dtype=torch.uint8, device="cuda")
    out = torch.empty_like(S)
    fb.focus_sinkhorn(shape, S, tau, iters, ws, out)
    torch.cuda.synchronize()
    ref = fo.sinkhorn(S[0].cpu().numpy().astype(np.float64), tau, iters)
    np.testing.assert_allclose(out[0].cpu().numpy(), ref, rtol=5e-4, atol=1e-7)
    np.testing.assert_allclose(out[0].sum(dim=0).cpu().numpy(), n / K, rtol=2e-2)      # groups close to balanced after 10 iterations
