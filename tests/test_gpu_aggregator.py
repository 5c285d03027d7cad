"""GPU parity of the aggregator-side steps: the second structured power iteration on the stacked factors
(Algorithm 1) and the effective rank (Sec. 3.3.1), against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from paper_2102_09631_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2102_09631_b200 import build, binding
    assert torch.cuda.is_available()
    build.build()
    binding.lib()
    return binding


def rel(x, ref):
    x = np.asarray(x, dtype=np.float64)
    return float(np.linalg.norm(x - ref) / max(np.linalg.norm(ref), 1e-300))


@pytest.mark.parametrize("K,h_in,h_out,r,iters", [
    (32, 784, 1024, 8, 3),     # config-2 first layer: S*r = 4*8 stacked rows reduced to 8 again
    (40, 512, 2048, 10, 2),    # config-3 ffn_up: 4 sites x r = 10
    (128, 768, 768, 16, 1),    # config-4 attention projection: 8 sites x 16
    (6, 40, 24, 8, 2),         # more directions asked for than the stacks hold: surplus rows are zero, result exact
])
def test_aggregate_compress_matches_oracle(oracle, B, K, h_in, h_out, r, iters):
    """The stacks are seeded fp32 factors (decaying strengths, like P carries sigma); both sides read the same bits."""
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(1000 + K)
    Pcat = torch.randn(K, h_in, generator=g) * (1.0 / torch.arange(1, K + 1)).unsqueeze(1)
    Qcat = torch.randn(K, h_out, generator=g) / (h_out ** 0.5)
    Q0 = torch.randn(r, h_out, generator=g)
    Ph = torch.empty(r, h_in, device=dev)
    Qh = torch.empty(r, h_out, device=dev)
    sg = torch.empty(r, device=dev)
    ws = B.new_workspace(B.dad_aggregate_workspace_bytes(h_in, h_out, K, r, iters), dev)
    B.dad_aggregate_compress(h_in, h_out, K, Pcat.to(dev), Qcat.to(dev), r, iters, Q0.to(dev), Ph, Qh, sg, ws)
    B.dad_check(ws)
    Po, Qo, so = oracle.aggregate_spi(Pcat, Qcat, Q0, iters)
    got = Ph.double().cpu().numpy().T @ Qh.double().cpu().numpy()
    assert rel(got, Po.T @ Qo) <= 1e-5
    live = [j for j in range(r) if np.any(Qo[j] != 0.0)]
    Qg = Qh.double().cpu().numpy()
    assert [j for j in range(r) if np.any(Qg[j] != 0.0)] == live
    assert np.linalg.norm(Qg[live] @ Qg[live].T - np.eye(len(live))) <= 1e-4
    assert np.allclose(sg.cpu().numpy(), np.linalg.norm(Ph.cpu().numpy(), axis=1), rtol=1e-5, atol=1e-30)
    if K <= r:
        full = oracle.reconstruct(Pcat, Qcat)
        assert rel(got, full) <= 1e-5


def test_two_stage_layer_end_to_end(oracle, B):
    """Algorithm 1 as printed: per-site SPI -> vertcat -> SPI of the stacks -> Phat^T Qhat, fp32 inputs."""
    dev = torch.device("cuda:0")
    S, N, h_in, h_out, r, iters = 4, 96, 160, 120, 6, 2
    A, D = wl.decaying_layer(S, N, h_in, h_out, 61, torch.float32)
    Q0 = wl.start_block(S, r, h_out, 61)
    Q0a = wl.start_block(1, r, h_out, 62)[0]
    plan = B.LayerPlan(A.to(dev), D.to(dev), r, iters)
    plan.step(A.to(dev), D.to(dev), Q0.to(dev))
    K = S * r
    Ph, Qh = torch.empty(r, h_in, device=dev), torch.empty(r, h_out, device=dev)
    ws = B.new_workspace(B.dad_aggregate_workspace_bytes(h_in, h_out, K, r, 2), dev)
    B.dad_aggregate_compress(h_in, h_out, K, plan.Pcat, plan.Qcat, r, 2, Q0a.to(dev), Ph, Qh, None, ws)
    grad_hat = torch.empty(h_in, h_out, device=dev)
    B.dad_reconstruct(h_in, h_out, r, Ph, Qh, grad_hat, B.DAD_F32, None)
    B.dad_check(ws)
    ref = oracle.two_stage_layer(A, D, Q0, iters, Q0a, 2)
    assert rel(grad_hat.double().cpu().numpy(), ref["grad_hat"]) <= 1e-5
    assert B.dad_bytes_rank(plan.layer, r) == ref["bytes_down"]   # what each site receives back
    # the broadcast estimate is a coarser approximation of the pooled gradient than the stacked one
    full = oracle.full_grad(A, D)
    assert rel(ref["grad_hat"], full) >= rel(ref["grad"], full) - 1e-12


def test_effective_rank_is_bit_exact(oracle, B):
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(5)
    S, r, h_in, h_out = 37, 16, 24, 40
    # strengths that decay at site-dependent rates, with exact ties to the threshold and zero sites mixed in
    sig = torch.rand(S, r, generator=g).sort(dim=1, descending=True).values * torch.logspace(0, -6, r).unsqueeze(0) ** \
        torch.rand(S, 1, generator=g)
    sig[3] = 0.0
    sig[5, 4] = sig[5, 0] * 1e-3
    sig[7, 1:] = 0.0
    for theta in (1e-3, 0.0, 0.25, 1.0):
        P = torch.randn(S, r, h_in, generator=g)
        Q = torch.randn(S, r, h_out, generator=g)
        Pd, Qd = P.to(dev), Q.to(dev)
        keep = torch.full((S,), -1, dtype=torch.int32, device=dev)
        L = B.dad_layer(S, 1, h_in, h_out, 0, h_in, h_out, h_in, h_out)
        B.dad_effective_rank(L, r, theta, sig.to(dev), keep, Pd, Qd)
        want = oracle.effective_rank(sig.numpy(), theta)
        assert np.array_equal(keep.cpu().numpy(), want)
        Pt, Qt = oracle.truncate(P, Q, want)
        assert np.array_equal(Pd.double().cpu().numpy(), Pt) and np.array_equal(Qd.double().cpu().numpy(), Qt)
        tx = [B.dad_bytes_rank(L, int(k)) if k > 0 else 0 for k in want]
        assert tx == [oracle.bytes_rank(int(k), h_in, h_out) if k > 0 else 0 for k in want]
    # factors may be left alone
    keep = torch.empty(S, dtype=torch.int32, device=dev)
    B.dad_effective_rank(L, r, 1e-3, sig.to(dev), keep, None, None)
    assert np.array_equal(keep.cpu().numpy(), oracle.effective_rank(sig.numpy(), 1e-3))


def test_effective_rank_drops_planted_noise_components(oracle, B):
    """A gradient of numerical rank 3 compressed with r = 6: both implementations keep 3 components per site,
    transmit half the bytes, and reconstruct the same gradient."""
    dev = torch.device("cuda:0")
    S, N, h_in, h_out, r, iters = 3, 50, 64, 48, 6, 4
    g = torch.Generator().manual_seed(9)
    A = torch.randn(S, N, h_in, generator=g)
    D = (torch.randn(S, N, 3, generator=g) * torch.tensor([1.0, 0.5, 0.25])) @ torch.randn(3, h_out, generator=g) \
        + 1e-7 * torch.randn(S, N, h_out, generator=g)
    Q0 = wl.start_block(S, r, h_out, 9)
    plan = B.LayerPlan(A.to(dev), D.to(dev), r, iters, zero_copy_gather=True)
    L = plan.layer
    B.dad_rank_compress(L, A.to(dev), D.to(dev), r, iters, Q0.to(dev), plan.P, plan.Q, plan.sigma, plan.ws)
    keep = torch.empty(S, dtype=torch.int32, device=dev)
    B.dad_effective_rank(L, r, 1e-3, plan.sigma, keep, plan.P, plan.Q)
    B.dad_reconstruct(h_in, h_out, S * r, plan.Pcat, plan.Qcat, plan.grads[0], B.DAD_F32, None)
    B.dad_check(plan.ws)
    Po, Qo, so = oracle.spi_block(A, D, Q0, iters)
    want = oracle.effective_rank(so.astype(np.float32), 1e-3)
    assert list(want) == [3] * S and np.array_equal(keep.cpu().numpy(), want)
    Pt, Qt = oracle.truncate(Po, Qo, want)
    ref = oracle.reconstruct(Pt.reshape(S * r, h_in), Qt.reshape(S * r, h_out))
    assert rel(plan.grads[0].double().cpu().numpy(), ref) <= 1e-5
    assert sum(B.dad_bytes_rank(L, int(k)) for k in keep.cpu()) * 2 == S * B.dad_bytes_rank(L, r)


@pytest.mark.parametrize("S,N,h_in,h_out,r,iters", [
    (2, 16, 64, 32, 4, 2),        # config 1
    (4, 64, 784, 1024, 8, 3),     # the paper's own setting: batch 64 per site, 784-1024-1024-10 MLP
    (4, 128, 1024, 1024, 8, 3),   # config-2 middle layer, N = 128 = the largest batch this form takes
    (3, 37, 200, 10, 8, 2),       # narrow output (r close to h_out), odd sizes
    (2, 5, 48, 40, 8, 1),         # batch smaller than r: exact, surplus vectors zero
])
def test_gram_form_matches_oracle_and_structured_form(oracle, B, S, N, h_in, h_out, r, iters):
    """dad_rank_compress_gram (C = A A^T precomputed, Algorithm 2 as printed) against the oracle's literal
    Algorithm 2 and against dad_rank_compress on the same inputs."""
    dev = torch.device("cuda:0")
    A, D = wl.decaying_layer(S, N, h_in, h_out, 400 + N, torch.float32)
    Q0 = wl.start_block(S, r, h_out, 400 + N)
    Ad, Dd, Q0d = A.to(dev), D.to(dev), Q0.to(dev)
    L = B.make_layer(Ad, Dd)
    P, Q, sg = (torch.empty(S, r, h_in, device=dev), torch.empty(S, r, h_out, device=dev), torch.empty(S, r, device=dev))
    ws = B.new_workspace(B.dad_rank_compress_gram_workspace_bytes(L, r, iters), dev)
    B.dad_rank_compress_gram(L, Ad, Dd, r, iters, Q0d, P, Q, sg, ws)
    B.dad_check(ws)
    Po, Qo, so = oracle.spi_gram(A, D, Q0, iters)
    P2, Q2, s2 = (torch.empty_like(P), torch.empty_like(Q), torch.empty_like(sg))
    ws2 = B.new_workspace(B.dad_workspace_bytes(L, r, iters), dev)
    B.dad_rank_compress(L, Ad, Dd, r, iters, Q0d, P2, Q2, s2, ws2)
    B.dad_check(ws2)
    Pn, Qn = P.double().cpu().numpy(), Q.double().cpu().numpy()
    for s in range(S):
        ref = Po[s].T @ Qo[s]
        assert rel(Pn[s].T @ Qn[s], ref) <= 1e-5
        assert rel(P2[s].double().cpu().numpy().T @ Q2[s].double().cpu().numpy(), ref) <= 1e-5
        live = [j for j in range(r) if np.any(Qo[s][j] != 0.0)]
        assert [j for j in range(r) if np.any(Qn[s][j] != 0.0)] == live
        assert np.linalg.norm(Qn[s][live] @ Qn[s][live].T - np.eye(len(live))) <= 1e-4
        scale = max(so[s].max(), 1e-300)
        assert np.abs(sg[s].cpu().numpy() - so[s]).max() <= 1e-5 * scale     # sqrt(v^T C v)
        assert np.abs(s2[s].cpu().numpy() - so[s]).max() <= 1e-5 * scale     # ||P_j||: the same number


def test_gram_form_refuses_what_it_does_not_take(B):
    dev = torch.device("cuda:0")
    A = torch.zeros(1, 129, 16, device=dev)
    D = torch.zeros(1, 129, 16, device=dev)
    L = B.make_layer(A, D)
    assert B.dad_rank_compress_gram_workspace_bytes(L, 4, 1) == 0
    buf = torch.empty(4, 16, device=dev)
    ws = B.new_workspace(1 << 20, dev)
    with pytest.raises(B.DadError, match="SHAPE"):
        B.dad_rank_compress_gram(L, A, D, 4, 1, buf, buf, buf, None, ws)
    Lb = B.make_layer(A[:, :64].bfloat16(), D[:, :64].bfloat16())
    with pytest.raises(B.DadError, match="DTYPE"):
        B.dad_rank_compress_gram(Lb, A, D, 4, 1, buf, buf, buf, None, ws)


@pytest.mark.gpu
@pytest.mark.parametrize("S,N,h_in,h_out,r,iters,dtype,raw", [
    (3, 40, 96, 72, 5, 3, torch.float32, True),
    (2, 300, 256, 512, 6, 2, torch.bfloat16, True),     # bf16 inputs through the general kernels, fp64 accumulation
    (2, 5, 48, 40, 8, 2, torch.float32, False),         # batch smaller than r: components beyond the rank carry nothing
])
def test_sequential_form_matches_the_oracles_algorithm_2(oracle, B, S, N, h_in, h_out, r, iters, dtype, raw):
    """dad_rank_compress_sequential (components one after the other, peel term, Sec. 3.3.1) against the oracle's
    vector-at-a-time Algorithm 2 on every site: projected gradient, and -- where the spectrum separates the
    components -- the vectors themselves, which the common start block fixes including their signs."""
    dev = torch.device("cuda:0")
    A, D = wl.decaying_layer(S, N, h_in, h_out, 700 + N, dtype, modes=8)
    Q0 = wl.start_block(S, r, h_out, 700 + N)
    Ad, Dd, Q0d = A.to(dev), D.to(dev), Q0.to(dev)
    L = B.make_layer(Ad, Dd)
    P, Q, sg = (torch.empty(S, r, h_in, device=dev), torch.empty(S, r, h_out, device=dev), torch.empty(S, r, device=dev))
    ws = B.new_workspace(B.dad_rank_compress_sequential_workspace_bytes(L, r, iters), dev)
    B.dad_rank_compress_sequential(L, Ad, Dd, r, iters, Q0d, P, Q, sg, ws)
    B.dad_check(ws)
    Pn, Qn, sn = P.double().cpu().numpy(), Q.double().cpu().numpy(), sg.double().cpu().numpy()
    for s in range(S):
        Po, Qo, so = oracle.spi_paper(A[s], D[s], Q0[s], iters)
        assert rel(Pn[s].T @ Qn[s], Po.T @ Qo) <= 1e-5
        if raw:
            assert rel(Qn[s], Qo) <= 1e-4 and rel(Pn[s], Po) <= 1e-4
            assert np.abs(sn[s] - so).max() <= 1e-5 * so.max()
            assert np.linalg.norm(Qn[s] @ Qn[s].T - np.eye(r)) <= 1e-5
