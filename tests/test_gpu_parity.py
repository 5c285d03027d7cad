"""Parity of the CUDA path (through the C ABI) with the float64 CPU oracle on the same seeded inputs.

Bars (relative Frobenius error): 1e-5 for fp32 inputs, 2e-2 for bf16 inputs with fp32 accumulation;
transmitted byte counts are bit-exact.  Any orthonormal basis of the subspace found gives the same
P_s^T Q_s, so parity is asserted on P_s^T Q_s, on the reconstructed gradient and on Q Q^T = I;
the raw factors are compared as well where the spectrum separates the vectors.
"""
import numpy as np
import pytest
import torch

from paper_2102_09631_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL = {torch.float32: 1e-5, torch.bfloat16: 2e-2}


@pytest.fixture(scope="module")
def B():
    from paper_2102_09631_b200 import build, binding
    assert torch.cuda.is_available(), "these tests need the B200"
    build.build()
    binding.lib()
    return binding


def rel(x, ref):
    x = np.asarray(x, dtype=np.float64)
    return float(np.linalg.norm(x - ref) / max(np.linalg.norm(ref), 1e-300))


GUARD_BYTES = 4096


class Guarded:
    """A device buffer with a band of 0xFF bytes (a NaN pattern for floats) before and after the part handed to the
    library: whatever the library writes outside its buffer shows up as a changed guard byte."""

    def __init__(self, nbytes, dev):
        self.n = int(nbytes)
        self.full = torch.full((self.n + 2 * GUARD_BYTES,), 0xFF, dtype=torch.uint8, device=dev)
        self.inner = self.full[GUARD_BYTES:GUARD_BYTES + self.n]

    def view(self, shape, dtype):
        return self.inner.view(dtype).view(shape)

    def intact(self):
        lo, hi = self.full[:GUARD_BYTES], self.full[GUARD_BYTES + self.n:]
        return bool((lo == 0xFF).all()) and bool((hi == 0xFF).all())


def guard_plan(B, plan, dev):
    """Moves every output and scratch buffer of a LayerPlan into guarded storage; returns the guards by name."""
    guards = {}

    def move(name, t):
        g = Guarded(t.numel() * t.element_size(), dev)
        guards[name] = g
        return g.view(t.shape, t.dtype)

    aliased = plan.Pcat.data_ptr() == plan.P.data_ptr()
    plan.P, plan.Q, plan.sigma = move("P", plan.P), move("Q", plan.Q), move("sigma", plan.sigma)
    if aliased:
        L = plan.layer
        plan.Pcat, plan.Qcat = plan.P.view(L.S * plan.r, L.h_in), plan.Q.view(L.S * plan.r, L.h_out)
    else:
        plan.Pcat, plan.Qcat = move("Pcat", plan.Pcat), move("Qcat", plan.Qcat)
    plan.grads = move("grad", plan.grads)
    plan.grad = plan.grads[0] if plan.groups == 1 else plan.grads
    plan.ws = move("ws", plan.ws)
    plan.ws[:256].zero_()        # the status words start out clear
    return guards


def run_gpu_layer(B, A, D, Q0, r, iters, math=None):
    """compress -> gather -> reconstruct and full_grad on the GPU; returns host float64 arrays.  Every buffer the
    library writes sits between guard bands, which must come back untouched."""
    dev = torch.device("cuda:0")
    Ad, Dd, Q0d = A.to(dev), D.to(dev), Q0.to(dev)
    plan = B.LayerPlan(Ad, Dd, r, iters)
    guards = guard_plan(B, plan, dev)
    if math is not None:
        plan.math = math
    plan.step(Ad, Dd, Q0d)
    gfull = Guarded(plan.grad.numel() * 4, dev)
    guards["full"] = gfull
    full = gfull.view(plan.grad.shape, torch.float32)
    tx_dad = B.bytes_array(plan.layer.S)
    B.dad_full_grad(plan.layer, Ad, Dd, full, tx_dad, plan.ws)
    B.dad_check(plan.ws)
    torch.cuda.synchronize()
    for name, g in guards.items():
        assert g.intact(), f"the library wrote outside its {name} buffer"
    f = lambda t: t.double().cpu().numpy()
    return dict(P=f(plan.P), Q=f(plan.Q), sigma=f(plan.sigma), Pcat=f(plan.Pcat), Qcat=f(plan.Qcat), grad=f(plan.grad),
                full=f(full), tx_rank=list(plan.bytes_tx), tx_dad=list(tx_dad), layer=plan.layer)


def check_layer(oracle, B, A, D, Q0, r, iters, tol, ortho_tol=1e-4, compare_factors=False):
    S, N, h_in = A.shape
    h_out = D.shape[2]
    g = run_gpu_layer(B, A, D, Q0, r, iters)
    o = oracle.rank_dad_layer(A, D, Q0, iters)
    e = A.element_size()
    # bytes: bit-exact
    assert g["tx_rank"] == [int(x) for x in o["bytes_tx"]] == [oracle.bytes_rank(r, h_in, h_out)] * S
    assert g["tx_dad"] == [oracle.bytes_dad(N, h_in, h_out, e)] * S
    # uncompressed dAD gradient
    assert rel(g["full"], oracle.full_grad(A, D)) <= tol
    # per-site projected gradients, orthonormality, sigma
    for s in range(S):
        ref = o["P"][s].T @ o["Q"][s]
        got = g["P"][s].T @ g["Q"][s]
        assert rel(got, ref) <= tol, (s, rel(got, ref))
        live = [j for j in range(r) if np.any(g["Q"][s][j] != 0.0)]
        live_o = [j for j in range(r) if np.any(o["Q"][s][j] != 0.0)]
        assert len(live) == len(live_o)
        Ql = g["Q"][s][live]
        if iters > 0:  # with no iteration Q is the caller's start block, returned as it came
            assert np.linalg.norm(Ql @ Ql.T - np.eye(len(live))) <= ortho_tol
        assert np.allclose(g["sigma"][s], np.linalg.norm(g["P"][s], axis=1), rtol=1e-5, atol=1e-30)
        if compare_factors:
            assert rel(g["Q"][s], o["Q"][s]) <= 50 * tol and rel(g["P"][s], o["P"][s]) <= 50 * tol
    # gather: stacks are the factors in site order, bit for bit
    assert np.array_equal(g["Pcat"], g["P"].reshape(S * r, h_in))
    assert np.array_equal(g["Qcat"], g["Q"].reshape(S * r, h_out))
    # reconstruction
    assert rel(g["grad"], o["grad"]) <= tol, rel(g["grad"], o["grad"])
    return g, o


@pytest.mark.parametrize("S,N,h_in,h_out,r,iters,dtype", [
    (2, 16, 64, 32, 4, 2, torch.float32),         # configuration 1
    (4, 128, 1024, 1024, 8, 3, torch.float32),    # configuration 2, hidden layer: 8 CTAs per site, 16 rows each
    (4, 128, 1024, 10, 8, 3, torch.float32),      # its output layer: fewer columns than CTAs in the cluster
    (18, 64, 784, 1024, 8, 3, torch.float32),     # the paper's own setting: batch 64 per site, 18 sites
    (1, 32, 784, 1024, 8, 3, torch.float32),      # the aggregator's stacks of a small layer as one site
    (3, 70, 264, 520, 40, 2, torch.float32),      # large rank (8 x 8 register blocks in the Cholesky-QR), ragged rows
    (5, 37, 50, 70, 7, 12, torch.float32),        # odd everything, many iterations
    (2, 100, 128, 256, 8, 2, torch.bfloat16),     # bf16 inputs small enough for one cluster: fp32 accumulation
    (3, 100, 70, 50, 7, 2, torch.bfloat16),
])
def test_one_launch_compress_matches_oracle_and_the_multi_launch_pipeline(oracle, B, S, N, h_in, h_out, r, iters, dtype):
    """Shapes the one-launch compress takes (a cluster per site for the whole structured power iteration):
    parity with the oracle at the usual bars, two runs bit for bit, and agreement with the multi-launch
    pipeline on the same inputs (same subspace: the projected gradients agree far inside the bar)."""
    dev = torch.device("cuda:0")
    seed = 900 + N + h_in
    A, D = wl.decaying_layer(S, N, h_in, h_out, seed, dtype)
    Q0 = wl.start_block(S, r, h_out, seed)
    path, C = B.dad_compress_path(B.make_layer(A.to(dev), D.to(dev)), r, iters)
    assert path in (B.DAD_PATH_FUSED, B.DAD_PATH_FUSED_L2) and C >= 1
    tol = TOL[dtype]
    g1, o = check_layer(oracle, B, A, D, Q0, r, iters, tol, ortho_tol=1e-3 if dtype == torch.bfloat16 else 1e-4)
    before = B.dad_launch_count()
    g2 = run_gpu_layer(B, A, D, Q0, r, iters)
    assert np.array_equal(g1["P"], g2["P"]) and np.array_equal(g1["Q"], g2["Q"]) and np.array_equal(g1["sigma"], g2["sigma"])
    B.dad_fused_enable(False)
    try:
        assert B.dad_compress_path(B.make_layer(A.to(dev), D.to(dev)), r, iters)[0] in (B.DAD_PATH_GENERAL, B.DAD_PATH_TENSOR, B.DAD_PATH_TENSOR_PAIRED)
        g3 = run_gpu_layer(B, A, D, Q0, r, iters)
    finally:
        B.dad_fused_enable(True)
    for s in range(S):
        assert rel(g1["P"][s].T @ g1["Q"][s], g3["P"][s].T @ g3["Q"][s]) <= tol
    assert rel(g1["grad"], g3["grad"]) <= tol


@pytest.mark.parametrize("S,N,h_in,h_out,r,iters,dtype", [(3, 40, 64, 48, 4, 2, torch.float32),      # one-launch, on chip
                                                          (3, 70, 264, 520, 40, 2, torch.float32),   # one-launch, through L2
                                                          (2, 300, 256, 512, 16, 2, torch.bfloat16),  # tensor-core pipeline
                                                          (3, 2000, 96, 40, 5, 1, torch.float32)])   # general pipeline
def test_q_may_alias_the_start_block(oracle, B, S, N, h_in, h_out, r, iters, dtype):
    """dad_rank_compress allows Q == Q0 (the start vectors are overwritten by the result): every pipeline gives,
    bit for bit, what it gives with separate buffers."""
    dev = torch.device("cuda:0")
    A, D = wl.decaying_layer(S, N, h_in, h_out, 61 + N, dtype, dev)
    Q0 = wl.start_block(S, r, h_out, 61 + N, dev)
    L = B.make_layer(A, D)
    ws = B.new_workspace(B.dad_workspace_bytes(L, r, iters), dev)
    P1, Q1 = torch.empty(S, r, h_in, device=dev), torch.empty(S, r, h_out, device=dev)
    sg1 = torch.empty(S, r, device=dev)
    B.dad_rank_compress(L, A, D, r, iters, Q0, P1, Q1, sg1, ws)
    B.dad_check(ws)
    P2, Q2, sg2 = torch.empty_like(P1), Q0.clone(), torch.empty_like(sg1)
    B.dad_rank_compress(L, A, D, r, iters, Q2, P2, Q2, sg2, ws)
    B.dad_check(ws)
    assert torch.equal(P1, P2) and torch.equal(Q1, Q2) and torch.equal(sg1, sg2)
    Po, Qo, _ = oracle.spi_block(A[:1].cpu(), D[:1].cpu(), Q0[:1].cpu(), iters)
    got = P2[0].double().cpu().numpy().T @ Q2[0].double().cpu().numpy()
    assert rel(got, Po[0].T @ Qo[0]) <= TOL[dtype]


def test_config1_single_linear_layer(oracle, B):
    cfg = wl.CONFIGS[1]
    A, D, Q0 = wl.layer_inputs(cfg, cfg.layers[0], 0)
    g, o = check_layer(oracle, B, A, D, Q0, cfg.r, cfg.iters, TOL[torch.float32])
    # "compare to full A^T D": the rank-4 estimate of a flat-spectrum gradient is far from it, equally
    # so for both implementations (an approximation error, not a parity criterion)
    err_gpu = rel(g["grad"], g["full"])
    err_ref = rel(o["grad"], oracle.full_grad(A, D))
    assert abs(err_gpu - err_ref) < 1e-5 and 0.3 < err_ref < 1.0


def test_config2_mlp_all_layers(oracle, B):
    cfg = wl.CONFIGS[2]
    mb = wl.mlp_layers(S=cfg.S, N=cfg.N)
    for i, shape in enumerate(cfg.layers):
        A, D = mb.A[i].float(), mb.D[i].float()
        assert A.shape == (cfg.S, cfg.N, shape.h_in) and D.shape == (cfg.S, cfg.N, shape.h_out)
        Q0 = wl.start_block(cfg.S, cfg.r, shape.h_out, wl.seed_for(2, i))
        check_layer(oracle, B, A, D, Q0, cfg.r, cfg.iters, TOL[torch.float32])


def test_config3_encoder_layer_projections(oracle, B):
    cfg = wl.CONFIGS[3]
    layers = wl.encoder_layers(S=cfg.S)
    seen = set()
    for i, (name, A, D) in enumerate(layers):
        if (A.shape[2], D.shape[2]) in seen and name != "o":
            continue  # q, k, v share a shape and an input; one of them and the output projection suffice
        seen.add((A.shape[2], D.shape[2]))
        assert A.dtype == torch.bfloat16 and A.shape[1] == cfg.N
        Q0 = wl.start_block(cfg.S, cfg.r, D.shape[2], wl.seed_for(3, i))
        check_layer(oracle, B, A, D, Q0, cfg.r, cfg.iters, TOL[torch.bfloat16], ortho_tol=1e-3)


@pytest.mark.parametrize("S,N,h_in,h_out,r,iters", [
    (4, 2048, 512, 2048, 10, 3),    # configuration 3's widest layer: 16 chunks fill tensor memory in one direction
    (16, 2048, 512, 512, 10, 2),    # its attention projections stacked as 16 slices: two shallow CTAs per SM
    (3, 1000, 200, 136, 7, 2),      # rows no multiple of 64 or 128, widths of no tile, rank below the padded 16
    (2, 100, 264, 520, 24, 2),      # one row block per site (nothing to sum), rank padded to 32
    (5, 333, 1024, 776, 32, 1),     # rank 32 at the widest X2 it takes (8 chunks of 64 columns of tensor memory)
    (2, 700, 768, 3072, 16, 2),     # paired in one direction only: the 3072-wide half keeps the two streaming kernels
])
def test_paired_launches_match_the_oracle_and_the_two_kernel_sequence(oracle, B, S, N, h_in, h_out, r, iters):
    """Calls of few row blocks can run each half of the operator of Eq. "reduced_iter" as one launch (Y stays on the SM;
    dad_pair_enable): parity with the oracle, two runs bit for bit (the partial blocks are summed in row-block order), and agreement with
    the two-kernel sequence on the same inputs far inside the bar."""
    dev = torch.device("cuda:0")
    seed = 3100 + N + h_out
    A, D = wl.decaying_layer(S, N, h_in, h_out, seed, torch.bfloat16)
    Q0 = wl.start_block(S, r, h_out, seed)
    L = B.make_layer(A.to(dev), D.to(dev))
    tol = TOL[torch.bfloat16]
    B.dad_fused_enable(False)    # the smallest of these sites would otherwise take the one-launch cluster form
    B.dad_pair_enable(True)      # the paired launches are an option (off by default: measured no faster, see the kernel's header)
    try:
        assert B.dad_compress_path(L, r, iters)[0] == B.DAD_PATH_TENSOR_PAIRED
        g1, o = check_layer(oracle, B, A, D, Q0, r, iters, tol, ortho_tol=1e-3)
        for s in range(S):
            assert rel(g1["P"][s].T @ g1["Q"][s], o["P"][s].T @ o["Q"][s]) <= 1e-4   # what the path delivers, not only the bar
        g2 = run_gpu_layer(B, A, D, Q0, r, iters)
        assert np.array_equal(g1["P"], g2["P"]) and np.array_equal(g1["Q"], g2["Q"]) and np.array_equal(g1["sigma"], g2["sigma"])
        B.dad_pair_enable(False)
        assert B.dad_compress_path(L, r, iters)[0] == B.DAD_PATH_TENSOR
        g3 = run_gpu_layer(B, A, D, Q0, r, iters)
    finally:
        B.dad_pair_enable(False)
        B.dad_fused_enable(True)
    for s in range(S):
        assert rel(g1["P"][s].T @ g1["Q"][s], g3["P"][s].T @ g3["Q"][s]) <= 1e-4
    assert rel(g1["grad"], g3["grad"]) <= 1e-4


@pytest.mark.parametrize("N,h_in,h_out,r,iters,dtype", [
    (6304 // 8, 768, 3072, 16, 3, torch.bfloat16),   # ViT-B ffn_up shape, ragged row count (788 = 6*128 + 20)
    (300, 1024, 1024, 4, 1, torch.bfloat16),          # GPT-2-medium attention projection, smallest sweep point
    (515, 4096, 1024, 64, 1, torch.bfloat16),         # ffn_down at the largest rank, odd row count
    (257, 200, 136, 10, 2, torch.bfloat16),           # widths that are multiples of 8 but of no tile
    (100, 70, 50, 7, 2, torch.bfloat16),              # widths that are not multiples of 8: general kernels
    (200, 256, 520, 24, 2, torch.bfloat16),           # ranks that pad to 3, 4, 5, 6, 7 row blocks of eight in the
    (200, 256, 512, 32, 2, torch.bfloat16),           # orthonormalisation (odd counts leave a middle block unpaired),
    (200, 512, 1024, 40, 2, torch.bfloat16),          # slabs of one to eight CTAs per site
    (200, 384, 776, 48, 1, torch.bfloat16),
    (200, 384, 768, 56, 1, torch.bfloat16),
    (260, 256, 4096, 64, 2, torch.bfloat16),          # widest slab at the largest rank, two iterations
    (130, 96, 40, 5, 3, torch.float32),
    (2048, 512, 256, 8, 2, torch.float32),            # recurrent layer 512 -> 256 over batch x time rows, fp32
    (72, 264, 2048, 48, 2, torch.float32),            # fp64 vectors, slab of the one-launch Cholesky-QR still fits
    (72, 264, 4096, 64, 1, torch.float32),            # fp64 vectors too wide for it: the multi-kernel Cholesky-QR
])
def test_shape_slices(oracle, B, N, h_in, h_out, r, iters, dtype):
    S = 2
    seed = 4242 + N + h_in
    A, D = wl.decaying_layer(S, N, h_in, h_out, seed, dtype)
    Q0 = wl.start_block(S, r, h_out, seed)
    check_layer(oracle, B, A, D, Q0, r, iters, TOL[dtype], ortho_tol=1e-3 if dtype == torch.bfloat16 else 1e-4)


@pytest.mark.parametrize("S,N,h_in,h_out", [
    (5, 1000, 520, 776),    # ragged 256 x 256 tiles, rows per site no multiple of a 64-row stage, split contraction
    (3, 1400, 256, 264),    # one full tile and a sliver
    (9, 512, 1024, 256),    # whole tiles, one stage-aligned site after the other
])
def test_full_grad_long_contraction(oracle, B, S, N, h_in, h_out):
    """The dAD gradient sum_s A_s^T D_s (Section 3.2) on the tensor cores where the contraction is long
    (S*N >= 4096 rows): bf16 products are exact in fp32, so only the fp32 accumulation order separates the
    result from the fp64 oracle -- a far tighter bar than the 2e-2 of the bf16 path as a whole."""
    dev = torch.device("cuda:0")
    A, D = wl.gaussian_layer(S, N, h_in, h_out, 77 + N, torch.bfloat16)
    L = B.make_layer(A.to(dev), D.to(dev))
    ws = B.new_workspace(B.dad_workspace_bytes(L, 1, 0), dev)
    grads = []
    for _ in range(2):
        grad = torch.full((h_in, h_out), float("nan"), device=dev)
        B.dad_full_grad(L, A.to(dev), D.to(dev), grad, None, ws)
        B.dad_check(ws)
        grads.append(grad.cpu())
    assert torch.equal(grads[0], grads[1])  # ordered split reduction: bit-identical runs
    assert rel(grads[0].double().numpy(), oracle.full_grad(A, D)) <= 1e-4


@pytest.mark.parametrize("S,groups,N,h_in,h_out,dtype", [
    (8, 4, 2048, 1024, 1024, torch.bfloat16),    # four 1024 x 1024 gradients: 64 tiles, split contraction, remainder CTAs
    (6, 3, 1500, 520, 264, torch.bfloat16),      # ragged tiles, rows no multiple of a stage, three products
    (4, 2, 300, 128, 96, torch.bfloat16),        # too small for the large tiles: one call per layer inside
    (4, 2, 64, 40, 24, torch.float32),           # fp32 inputs: the FMA kernel, one call per layer inside
])
def test_full_grad_of_several_stacked_layers_in_one_call(oracle, B, S, groups, N, h_in, h_out, dtype):
    """dad_full_grad_grouped: layer g owns slices g*S' .. of A and D; every gradient against the oracle on its own
    slices, against dad_full_grad on the same slices, two runs bit for bit, guard bands around the output intact."""
    dev = torch.device("cuda:0")
    A, D = wl.gaussian_layer(S, N, h_in, h_out, 515 + N, dtype, dev)
    L = B.make_layer(A, D)
    ws = B.new_workspace(max(256, B.dad_full_grad_grouped_workspace_bytes(L, groups)), dev)
    Sg = S // groups
    outs = []
    for _ in range(2):
        guard = Guarded(groups * h_in * h_out * 4, dev)
        grads = guard.view((groups, h_in, h_out), torch.float32)
        tx = B.bytes_array(S)
        B.dad_full_grad_grouped(L, groups, A, D, grads, tx, ws)
        B.dad_check(ws)
        torch.cuda.synchronize()
        assert guard.intact()
        outs.append(grads.clone())
    assert torch.equal(outs[0], outs[1])
    assert list(tx) == [oracle.bytes_dad(N, h_in, h_out, A.element_size())] * S
    tol = 1e-4 if dtype == torch.bfloat16 else 1e-5
    for g in range(groups):
        sl = slice(g * Sg, (g + 1) * Sg)
        ref = oracle.full_grad(A[sl].cpu(), D[sl].cpu())
        assert rel(outs[0][g].double().cpu().numpy(), ref) <= tol, g
        L1 = B.make_layer(A[sl], D[sl])
        ws1 = B.new_workspace(max(256, B.dad_workspace_bytes(L1, 1, 0)), dev)
        one = torch.empty(h_in, h_out, device=dev)
        B.dad_full_grad(L1, A[sl], D[sl], one, None, ws1)
        B.dad_check(ws1)
        assert rel(outs[0][g].double().cpu().numpy(), one.double().cpu().numpy()) <= tol
    with pytest.raises(Exception):
        B.dad_full_grad_grouped(L, S + 1, A, D, outs[0], None, ws)     # does not divide the slices


@pytest.mark.parametrize("h_in,h_out", [(512, 5120), (520, 5000)])   # whole tiles; ragged last tile row and column
def test_full_grad_with_remainder_ctas(oracle, B, h_in, h_out):
    """40 tiles of 256 x 256 in 3 splits leave 28 SMs without a CTA; those take the tail of every tile's contraction,
    two tiles each in turn (a fourth partial tile per output tile).  Sampled output rows against the oracle, and two
    runs bit for bit."""
    dev = torch.device("cuda:0")
    S, N = 5, 6144     # 480 blocks of 64 rows; 40 tiles: 3 x 142 blocks in the main part, 54 in the tail (60 tiles: 2 x 215, 50)
    A, D = wl.gaussian_layer(S, N, h_in, h_out, 4111, torch.bfloat16, dev)
    L = B.make_layer(A, D)
    ws = B.new_workspace(B.dad_workspace_bytes(L, 1, 0), dev)
    grads = []
    for _ in range(2):
        grad = torch.full((h_in, h_out), float("nan"), device=dev)
        B.dad_full_grad(L, A, D, grad, None, ws)
        B.dad_check(ws)
        grads.append(grad.cpu())
    assert torch.equal(grads[0], grads[1])
    rows = [0, 255, 256, 300, h_in - 1]
    ref = oracle.full_grad(A[:, :, rows].cpu(), D.cpu())
    assert rel(grads[0][rows].double().numpy(), ref) <= 1e-4


@pytest.mark.parametrize("h_in,h_out,K,batch", [(1024, 1024, 256, 16), (264, 520, 40, 3), (70, 50, 12, 2),
                                                (520, 5000, 40, 6),     # 600 tiles, ragged last tile row and column:
                                                (2048, 4104, 72, 1)])   # the persistent kernel, batched and single
def test_reconstruct_batched_is_the_per_layer_sum_of_outer_products(oracle, B, h_in, h_out, K, batch):
    """Algorithm 1's P^T Q step for several layers of one shape in one call: every entry against the oracle's
    sum of outer products over its own K rows of the stacks, and batch = 1 against dad_reconstruct bit for bit."""
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(1000 + K)
    Pcat = torch.randn(batch * K, h_in, generator=g)
    Qcat = torch.randn(batch * K, h_out, generator=g)
    for math, tol in ((B.DAD_F32, 1e-5), (B.DAD_BF16, 1e-4)):
        ws = B.new_workspace(B.dad_reconstruct_batched_workspace_bytes(h_in, h_out, K, batch, math), dev)
        grads = torch.full((batch, h_in, h_out), float("nan"), device=dev)
        B.dad_reconstruct_batched(h_in, h_out, K, batch, Pcat.to(dev), Qcat.to(dev), grads, math, ws)
        B.dad_check(ws)
        for b in range(batch):
            rows = slice(b * K, (b + 1) * K)
            ref = oracle.reconstruct(Pcat[rows], Qcat[rows])
            assert rel(grads[b].double().cpu().numpy(), ref) <= tol, (b, math)
        one, single = torch.empty(h_in, h_out, device=dev), torch.empty(h_in, h_out, device=dev)
        B.dad_reconstruct_batched(h_in, h_out, K, 1, Pcat.to(dev), Qcat.to(dev), one, math, ws)
        B.dad_reconstruct(h_in, h_out, K, Pcat.to(dev), Qcat.to(dev), single, math, ws)
        assert torch.equal(one, single)


@pytest.mark.parametrize("h_in,h_out,K,batch", [(1024, 4096, 1024, 1), (1024, 1024, 256, 4), (264, 520, 40, 3)])
def test_one_term_reconstruction_stays_inside_the_contract(oracle, B, h_in, h_out, K, batch):
    """DAD_BF16_1TERM multiplies the bf16 roundings of the factors once: a third of the work of the three-term
    product, 8 significant bits of each factor.  Against the oracle's sum of outer products the error is a few
    1e-3 -- inside the 2e-2 bar of bf16 arithmetic, and pinned here at 6e-3 so that a further loss shows."""
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(5150 + K)
    Pcat = torch.randn(batch * K, h_in, generator=g)
    Qcat = torch.randn(batch * K, h_out, generator=g)
    ws = B.new_workspace(B.dad_reconstruct_batched_workspace_bytes(h_in, h_out, K, batch, B.DAD_BF16_1TERM), dev)
    assert ws.numel() <= max(256, B.dad_reconstruct_batched_workspace_bytes(h_in, h_out, K, batch, B.DAD_BF16))
    grads = torch.full((batch, h_in, h_out), float("nan"), device=dev)
    B.dad_reconstruct_batched(h_in, h_out, K, batch, Pcat.to(dev), Qcat.to(dev), grads, B.DAD_BF16_1TERM, ws)
    B.dad_check(ws)
    rows = [0, 1, h_in // 2, h_in - 1]
    for b in range(batch):
        sl = slice(b * K, (b + 1) * K)
        ref = oracle.reconstruct(Pcat[sl][:, rows], Qcat[sl])
        err = rel(grads[b][rows].double().cpu().numpy(), ref)
        assert 1e-4 < err <= 6e-3, (b, err)      # it really is the one-term product, and no worse than that


def test_factors_match_on_separated_spectrum(oracle, B):
    """With well separated singular values and enough iterations each vector is determined up to
    rounding (thin QR with positive diagonal fixes the sign), so the raw factors agree too."""
    S, N, h_in, h_out, r = 2, 64, 48, 40, 3
    A, D = wl.decaying_layer(S, N, h_in, h_out, 99, torch.float32, modes=6, noise=0.0)
    Q0 = wl.start_block(S, r, h_out, 99)
    check_layer(oracle, B, A, D, Q0, r, 12, 1e-5, compare_factors=True)


def test_rank_exceeding_true_rank_is_exact(oracle, B):
    """r >= rank(A_s^T D_s): the estimate reproduces the uncompressed gradient, surplus vectors are zero."""
    S, N, h_in, h_out, r = 3, 5, 64, 48, 8   # batch of 5 rows: rank <= 5 < r
    A, D = wl.gaussian_layer(S, N, h_in, h_out, 7)
    Q0 = wl.start_block(S, r, h_out, 7)
    g, o = check_layer(oracle, B, A, D, Q0, r, 1, 1e-5)
    assert rel(g["grad"], g["full"]) <= 1e-5
    for s in range(S):
        assert sum(1 for j in range(r) if np.all(g["Q"][s][j] == 0.0)) == r - N
        assert np.all(g["sigma"][s][N:] == 0.0)


@pytest.mark.parametrize("iters,dependent_start", [(2, False), (1, True)])
def test_many_sites_at_large_rank(oracle, B, iters, dependent_start):
    """320 sites at r = 32: more CTAs than the GPU holds at once, so the orthonormalisation takes its two-launch
    form (Gram + one factorisation per site, then the substitution).  With two start vectors that repeat others
    (one of them scaled) the iterate has two exactly dependent vectors: their pivots reach the floor, the second
    pass runs, and those two come out as zeros -- in the oracle too, so the live sets must agree."""
    S, N, h_in, h_out, r = 320, 72, 128, 256, 32
    A, D = wl.gaussian_layer(S, N, h_in, h_out, 587, torch.bfloat16)
    Q0 = wl.start_block(S, r, h_out, 587)
    if dependent_start:
        Q0[:, r - 1] = Q0[:, 0]
        Q0[:, 9] = 2.0 * Q0[:, 4]
    g, o = check_layer(oracle, B, A, D, Q0, r, iters, TOL[torch.bfloat16], ortho_tol=1e-3)
    if dependent_start:
        for s in (0, 77, S - 1):
            assert [j for j in range(r) if np.all(g["Q"][s][j] == 0.0)] == [9, r - 1]


@pytest.mark.parametrize("S,N,h_in,h_out,r,iters", [
    (80, 200, 520, 768, 40, 2),     # ragged second row tile, 520 columns = 4 tiles and a sliver
    (75, 512, 256, 1024, 64, 1),    # whole tiles everywhere
    (90, 250, 1024, 136, 56, 2),    # a 136-wide operand: one tile and eight columns
])
def test_many_sites_above_rank_32(oracle, B, S, N, h_in, h_out, r, iters):
    """Ranks that pad to 64 on launches of more than one wave of CTAs (the shallow two- and three-stage forms of the thin
    products, 128-column accumulators), with ragged row and column tiles.  Parity with the oracle on every site at the
    accuracy the path delivers, and two runs bit for bit."""
    A, D = wl.decaying_layer(S, N, h_in, h_out, 7300 + N, torch.bfloat16)
    Q0 = wl.start_block(S, r, h_out, 7300 + N)
    g1, o = check_layer(oracle, B, A, D, Q0, r, iters, TOL[torch.bfloat16], ortho_tol=1e-3)
    for s in range(S):
        assert rel(g1["P"][s].T @ g1["Q"][s], o["P"][s].T @ o["Q"][s]) <= 1e-4
    g2 = run_gpu_layer(B, A, D, Q0, r, iters)
    assert np.array_equal(g1["P"], g2["P"]) and np.array_equal(g1["Q"], g2["Q"])


def test_edge_shapes(oracle, B):
    # one row, one site, r = 1; r = min(h); zero iterations; strided (non-contiguous) rows and sites
    A, D = wl.gaussian_layer(1, 1, 8, 8, 1)
    check_layer(oracle, B, A, D, wl.start_block(1, 1, 8, 1), 1, 2, 1e-5)
    A, D = wl.gaussian_layer(2, 40, 16, 6, 2)
    check_layer(oracle, B, A, D, wl.start_block(2, 6, 6, 2), 6, 2, 1e-5)
    check_layer(oracle, B, A, D, wl.start_block(2, 3, 6, 3), 3, 0, 1e-5)
    Abig, Dbig = wl.gaussian_layer(3, 50, 40, 24, 3)
    A, D = Abig[:, :33, :32], Dbig[:, :33, :16]   # views: ld > h, site stride > N*ld
    assert not A.is_contiguous()
    dev = torch.device("cuda:0")
    Ad, Dd = Abig.to(dev)[:, :33, :32], Dbig.to(dev)[:, :33, :16]
    Q0 = wl.start_block(3, 4, 16, 4)
    plan = B.LayerPlan(Ad, Dd, 4, 2)
    assert plan.layer.ldA == 40 and plan.layer.strideA == 50 * 40
    plan.step(Ad, Dd, Q0.to(dev))
    B.dad_check(plan.ws)
    o = oracle.rank_dad_layer(A.contiguous(), D.contiguous(), Q0, 2)
    assert rel(plan.grad.double().cpu().numpy(), o["grad"]) <= 1e-5


def test_zero_copy_gather_and_determinism(oracle, B):
    dev = torch.device("cuda:0")
    A, D = wl.decaying_layer(4, 700, 256, 512, 11, torch.bfloat16)
    Q0 = wl.start_block(4, 16, 512, 11)
    Ad, Dd, Q0d = A.to(dev), D.to(dev), Q0.to(dev)
    outs = []
    for zero_copy in (False, True, True):
        plan = B.LayerPlan(Ad, Dd, 16, 2, zero_copy_gather=zero_copy)
        plan.step(Ad, Dd, Q0d)
        B.dad_check(plan.ws)
        outs.append((plan.grad.clone(), plan.P.clone(), plan.Q.clone()))
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a, b)          # aliasing the stacks changes nothing
    for a, b in zip(outs[1], outs[2]):
        assert torch.equal(a, b)          # two runs agree bit for bit


def test_nan_input_is_reported_not_trapped(B):
    dev = torch.device("cuda:0")
    A, D = wl.gaussian_layer(1, 32, 16, 16, 5)
    D[0, 3, 2] = float("nan")
    plan = B.LayerPlan(A.to(dev), D.to(dev), 4, 1)
    plan.step(A.to(dev), D.to(dev), wl.start_block(1, 4, 16, 5).to(dev))
    with pytest.raises(B.DadError, match="NUMERIC"):
        B.dad_check(plan.ws)
    # the context is intact: a clean call afterwards succeeds
    A, D = wl.gaussian_layer(1, 32, 16, 16, 6)
    plan = B.LayerPlan(A.to(dev), D.to(dev), 4, 1)
    plan.step(A.to(dev), D.to(dev), wl.start_block(1, 4, 16, 6).to(dev))
    B.dad_check(plan.ws)


def test_bounded_wait_runs_out_reports_timeout_and_leaves_the_context_usable(oracle, B):
    """The give-up path of the tensor-core kernels, exercised without hanging or faulting anything: a small tile
    whose multiplying role expects one block more than is loaded, with a limit of 1024 polls.  The wait runs out,
    the CTA drains what it issued, frees its tensor memory and returns; the status word says DAD_ERR_TIMEOUT; an
    ordinary call on the same workspace afterwards is clean and correct."""
    dev = torch.device("cuda:0")
    S, N, h_in, h_out, r, iters = 2, 300, 256, 512, 16, 2
    A, D = wl.decaying_layer(S, N, h_in, h_out, 5, torch.bfloat16)
    Q0 = wl.start_block(S, r, h_out, 5)
    Ad, Dd, Q0d = A.to(dev), D.to(dev), Q0.to(dev)
    plan = B.LayerPlan(Ad, Dd, r, iters)
    assert plan.ws.numel() >= B.DAD_SELFTEST_BYTES
    for _ in range(2):
        B.dad_selftest_bounded_wait(plan.ws)
        with pytest.raises(B.DadError, match="TIMEOUT"):
            B.dad_check(plan.ws)
        plan.step(Ad, Dd, Q0d)
        B.dad_check(plan.ws)                       # the status word was cleared by the call; nothing else is reported
        o = oracle.rank_dad_layer(A, D, Q0, iters)
        assert rel(plan.grad.double().cpu().numpy(), o["grad"]) <= 1e-4


def test_reconstruct_and_full_grad_at_full_size_on_sampled_rows(oracle, B):
    """Largest shapes of the GPT-2-medium configuration; the oracle computes sampled output rows."""
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(31)
    h_in, h_out, K = 1024, 4096, 1024
    Pcat = torch.randn(K, h_in, generator=g)
    Qcat = torch.randn(K, h_out, generator=g)
    rows = [0, 1, 63, 64, 517, 1023]
    for math in (B.DAD_F32, B.DAD_BF16):
        grad = torch.empty(h_in, h_out, device=dev)
        ws = B.new_workspace(B.dad_reconstruct_workspace_bytes(h_in, h_out, K, math), dev)
        B.dad_reconstruct(h_in, h_out, K, Pcat.to(dev), Qcat.to(dev), grad, math, ws)
        ref = oracle.reconstruct(Pcat[:, rows], Qcat)
        # tensor-core reconstruction multiplies two-term bf16 splits (three products): ~2^-16 relative
        assert rel(grad[rows].double().cpu().numpy(), ref) <= (1e-5 if math == B.DAD_F32 else 1e-4)
    S, N = 16, 4096
    A, D = wl.decaying_layer(S, N, h_in, h_out, 32, torch.bfloat16, device=dev)
    L = B.make_layer(A, D)
    grad = torch.empty(h_in, h_out, device=dev)
    ws = B.new_workspace(B.dad_workspace_bytes(L, 1, 0), dev)
    B.dad_full_grad(L, A, D, grad, None, ws)
    torch.cuda.synchronize()
    ref = oracle.full_grad(A[:, :, rows].cpu(), D.cpu())
    assert rel(grad[rows].double().cpu().numpy(), ref) <= 2e-2


def test_compress_at_full_size_on_sampled_sites(oracle, B):
    """GPT-2-medium ffn_up layer exactly as the benchmark launches it (S=16, N=4096, r=16, 3 iterations);
    sites are independent, so the oracle recomputes two of them from the same inputs."""
    dev = torch.device("cuda:0")
    cfg = wl.CONFIGS[5]
    shape = cfg.layers[1]
    A, D, Q0 = wl.layer_inputs(cfg, shape, 1, device=dev)
    plan = B.LayerPlan(A, D, cfg.r, cfg.iters)
    plan.step(A, D, Q0)
    B.dad_check(plan.ws)
    sites = [0, 11]
    Po, Qo, _ = oracle.spi_block(A[sites].cpu(), D[sites].cpu(), Q0[sites].cpu(), cfg.iters)
    for i, s in enumerate(sites):
        got = plan.P[s].double().cpu().numpy().T @ plan.Q[s].double().cpu().numpy()
        assert rel(got, Po[i].T @ Qo[i]) <= ACCURACY_BAR   # the contract says 2e-2; what is delivered is pinned too
        Qg = plan.Q[s].double().cpu().numpy()
        assert np.linalg.norm(Qg @ Qg.T - np.eye(cfg.r)) <= 1e-3
    assert list(plan.bytes_tx) == [oracle.bytes_rank(cfg.r, shape.h_in, shape.h_out)] * cfg.S


ACCURACY_BAR = 1e-4   # delivered accuracy of the bf16 path on these workloads is a few 1e-6: losing a plane would show


def full_size_case(oracle, B, cfg_index, shape, r, iters, groups, sites, whole_layer=None):
    """One call exactly as the benchmark launches it (same-shape layers of `groups` blocks stacked as extra slices);
    the oracle recomputes the sampled sites and, if asked, one whole layer's reconstructed gradient."""
    dev = torch.device("cuda:0")
    cfg = wl.CONFIGS[cfg_index]
    S = cfg.S
    A, D = wl.decaying_layer(S * groups, cfg.N, shape[0], shape[1], 7000 + cfg_index * 10 + r, torch.bfloat16, device=dev)
    Q0 = wl.start_block(S * groups, r, shape[1], 7000 + r, dev)
    plan = B.LayerPlan(A, D, r, iters, groups=groups)
    guards = guard_plan(B, plan, dev)
    grads = plan.step(A, D, Q0)
    B.dad_check(plan.ws)
    for name, g in guards.items():
        assert g.intact(), f"the library wrote outside its {name} buffer"
    Po, Qo, _ = oracle.spi_block(A[sites].cpu(), D[sites].cpu(), Q0[sites].cpu(), iters)
    for i, s in enumerate(sites):
        got = plan.P[s].double().cpu().numpy().T @ plan.Q[s].double().cpu().numpy()
        err = rel(got, Po[i].T @ Qo[i])
        assert err <= ACCURACY_BAR, (s, err)
        Qg = plan.Q[s].double().cpu().numpy()
        assert np.linalg.norm(Qg @ Qg.T - np.eye(r)) <= 1e-3
    assert list(plan.bytes_tx) == [oracle.bytes_rank(r, shape[0], shape[1])] * (S * groups)
    if whole_layer is not None:
        sl = slice(whole_layer * S, (whole_layer + 1) * S)
        o = oracle.rank_dad_layer(A[sl].cpu(), D[sl].cpu(), Q0[sl].cpu(), iters)
        g = grads[whole_layer] if groups > 1 else grads
        err = rel(g.double().cpu().numpy(), o["grad"])
        assert err <= ACCURACY_BAR, err


def test_vit_b_configuration_at_its_own_size(oracle, B):
    """Configuration 4 as the benchmark launches it: N = 6304 rows per site (49 row tiles of 128 and a 32-row
    remainder), S = 8, r = 16, three iterations -- the attention projections of a block stacked in one call
    (768 CTAs in the column products: their five-stage form), and one 768 -> 3072 layer."""
    cfg = wl.CONFIGS[4]
    assert (cfg.N, cfg.S, cfg.r) == (6304, 8, 16)
    full_size_case(oracle, B, 4, (768, 768), cfg.r, cfg.iters, groups=4, sites=[0, 29], whole_layer=2)
    full_size_case(oracle, B, 4, (768, 3072), cfg.r, cfg.iters, groups=1, sites=[3, 7])


@pytest.mark.parametrize("shape,r,iters,groups", [((4096, 1024), 16, 3, 1),     # the down projection at full size
                                                  ((1024, 1024), 4, 1, 16),     # the sweep's smallest rank, stacked call
                                                  ((1024, 4096), 4, 3, 4)])
def test_gpt2_medium_configuration_remaining_shapes_at_full_size(oracle, B, shape, r, iters, groups):
    full_size_case(oracle, B, 5, shape, r, iters, groups, sites=[1, 16 * groups - 1])


@pytest.mark.parametrize("r,iters", [(16, 3), (64, 1)])
def test_stacked_call_at_the_benchmarks_launch_shape(oracle, B, r, iters):
    """The call the benchmark times for the attention projections of the GPT-2-medium configuration: the
    1024 -> 1024 layers of four consecutive blocks stacked as 16 x 16 = 256 slices of one call, i.e. 2048-CTA
    launches of both thin products and the batched reconstruction; at r = 16 (three iterations) the one-wave
    Cholesky-QR, at r = 64 (the sweep's largest rank) its two-launch form over 256 sites.  The oracle recomputes
    three sampled sites and, for one whole layer of the stack, the reconstructed gradient from the same inputs."""
    dev = torch.device("cuda:0")
    cfg = wl.CONFIGS[5]
    S, groups = cfg.S, 16
    shape = cfg.layers[0]
    assert (shape.h_in, shape.h_out) == (1024, 1024)
    A, D = wl.decaying_layer(S * groups, cfg.N, shape.h_in, shape.h_out, 9051, torch.bfloat16, device=dev)
    Q0 = wl.start_block(S * groups, r, shape.h_out, 9051, dev)
    plan = B.LayerPlan(A, D, r, iters, groups=groups)
    grads = plan.step(A, D, Q0)
    B.dad_check(plan.ws)
    sites = [0, 101, S * groups - 1]
    Po, Qo, _ = oracle.spi_block(A[sites].cpu(), D[sites].cpu(), Q0[sites].cpu(), iters)
    for i, s in enumerate(sites):
        got = plan.P[s].double().cpu().numpy().T @ plan.Q[s].double().cpu().numpy()
        assert rel(got, Po[i].T @ Qo[i]) <= ACCURACY_BAR
        Qg = plan.Q[s].double().cpu().numpy()
        assert np.linalg.norm(Qg @ Qg.T - np.eye(r)) <= 1e-3
    g = 6                                   # one whole layer of the stack: its 16 sites and its gradient
    sl = slice(g * S, (g + 1) * S)
    o = oracle.rank_dad_layer(A[sl].cpu(), D[sl].cpu(), Q0[sl].cpu(), iters)
    assert rel(grads[g].double().cpu().numpy(), o["grad"]) <= ACCURACY_BAR
    assert list(plan.bytes_tx)[sl] == [int(x) for x in o["bytes_tx"]]


def test_stacked_layers_match_separate_calls(oracle, B):
    """Several layers of one shape stacked as extra slices of one call (groups > 1) give, layer by layer,
    what separate calls give (up to the order of the split sums) and agree with the oracle."""
    dev = torch.device("cuda:0")
    S, groups, N, h_in, h_out, r, iters = 3, 2, 200, 128, 192, 8, 2
    A, D = wl.decaying_layer(S * groups, N, h_in, h_out, 77, torch.bfloat16)
    Q0 = wl.start_block(S * groups, r, h_out, 77)
    Ad, Dd, Q0d = A.to(dev), D.to(dev), Q0.to(dev)
    plan = B.LayerPlan(Ad, Dd, r, iters, groups=groups)
    grads = plan.step(Ad, Dd, Q0d).clone()
    B.dad_check(plan.ws)
    assert grads.shape == (groups, h_in, h_out)
    for g in range(groups):
        sl = slice(g * S, (g + 1) * S)
        single = B.LayerPlan(Ad[sl], Dd[sl], r, iters)
        single.step(Ad[sl], Dd[sl], Q0d[sl])
        B.dad_check(single.ws)
        # the row splits of the column products depend on the slice count, so sums are ordered differently
        assert rel(single.grad.double().cpu().numpy(), grads[g].double().cpu().numpy()) <= 1e-3
        ref = oracle.rank_dad_layer(A[sl], D[sl], Q0[sl], iters)
        assert rel(grads[g].double().cpu().numpy(), ref["grad"]) <= TOL[torch.bfloat16]
    assert list(plan.bytes_tx) == [oracle.bytes_rank(r, h_in, h_out)] * (S * groups)


def test_reconstruction_deferred_to_one_batched_call(oracle, B):
    """A plan of several calls (LayerPlan(calls=3)): every call compresses and gathers into its own slot, finish()
    reconstructs the layers of all slots in one batched call.  Bit for bit what per-call plans give, and one layer
    against the oracle."""
    dev = torch.device("cuda:0")
    S, N, h_in, h_out, r, iters, groups, calls = 3, 260, 512, 768, 8, 2, 2, 3
    sets = []
    for c in range(calls):
        A, D = wl.decaying_layer(S * groups, N, h_in, h_out, 8800 + c, torch.bfloat16, device=dev)
        sets.append((A, D, wl.start_block(S * groups, r, h_out, 8800 + c, dev)))
    plan = B.LayerPlan(*sets[0][:2], r, iters, groups=groups, calls=calls)
    for c, (A, D, Q0) in enumerate(sets):
        plan.step(A, D, Q0, call=c)
    grads = plan.finish()
    B.dad_check(plan.ws)
    B.dad_check(plan.ws_all)
    single = B.LayerPlan(*sets[0][:2], r, iters, groups=groups)
    for c, (A, D, Q0) in enumerate(sets):
        g = single.step(A, D, Q0)
        assert torch.equal(g, grads[c * groups:(c + 1) * groups])
        assert torch.equal(single.P, plan.P_all[c]) and torch.equal(single.Q, plan.Q_all[c])
    A, D, Q0 = sets[1]
    o = oracle.rank_dad_layer(A[S:2 * S].cpu(), D[S:2 * S].cpu(), Q0[S:2 * S].cpu(), iters)   # call 1, second layer
    assert rel(grads[1 * groups + 1].double().cpu().numpy(), o["grad"]) <= ACCURACY_BAR


def test_host_entry_point_matches_device_path_and_oracle(oracle, B):
    """dad_rank_dad_host: inputs in (pinned) host memory, gradient back in host memory; same result as the
    three device calls, bit for bit, for dense and for strided host layouts."""
    dev = torch.device("cuda:0")
    S, N, h_in, h_out, r, iters = 3, 260, 128, 192, 8, 2
    for dtype, tol in ((torch.bfloat16, 2e-2), (torch.float32, 1e-5)):
        Abig, Dbig = wl.decaying_layer(S, N + 7, h_in + 8, h_out + 16, 55, dtype)
        Q0 = wl.start_block(S, r, h_out, 55).pin_memory()
        for strided in (False, True):
            if strided:
                A, D = Abig.pin_memory()[:, :N, :h_in], Dbig.pin_memory()[:, :N, :h_out]
            else:
                A, D = Abig[:, :N, :h_in].contiguous().pin_memory(), Dbig[:, :N, :h_out].contiguous().pin_memory()
            L = B.make_layer(A, D)
            assert (L.ldA == h_in) == (not strided)
            math = L.dtype
            scratch = torch.empty(B.dad_rank_dad_host_scratch_bytes(L, r, iters, math), dtype=torch.uint8, device=dev)
            grad_host = torch.full((h_in, h_out), float("nan")).pin_memory()
            tx = B.bytes_array(S)
            B.dad_rank_dad_host(L, A, D, Q0, r, iters, math, grad_host, scratch, tx)
            torch.cuda.synchronize()
            Ad, Dd = A.contiguous().to(dev), D.contiguous().to(dev)
            plan = B.LayerPlan(Ad, Dd, r, iters, zero_copy_gather=True)
            plan.step(Ad, Dd, Q0.to(dev))
            B.dad_check(plan.ws)
            assert torch.equal(plan.grad.cpu(), grad_host)
            ref = oracle.rank_dad_layer(A.contiguous(), D.contiguous(), Q0, iters)
            assert rel(grad_host.double().numpy(), ref["grad"]) <= tol
            assert list(tx) == [int(x) for x in ref["bytes_tx"]]
    # host-detectable errors come back before anything is queued
    E = B.STATUS_NAMES.index
    small = torch.empty(256, dtype=torch.uint8, device=dev)
    with pytest.raises(B.DadError, match="WORKSPACE"):
        B.dad_rank_dad_host(L, A, D, Q0, r, iters, math, grad_host, small)
    assert B.dad_rank_dad_host_scratch_bytes(L, 0, iters, math) == 0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_degenerate_inputs(oracle, B, dtype):
    """The degenerate cases of the method: no signal at all (zero errors), identical start vectors (a start
    block of rank 1), and a single repeated row (a rank-1 gradient compressed with r = 4)."""
    tol = TOL[dtype]
    S, N, h_in, h_out, r = 2, 136, 64, 72, 4
    A, D = wl.gaussian_layer(S, N, h_in, h_out, 31, dtype)
    Q0 = wl.start_block(S, r, h_out, 31)
    # (a) zero errors: every vector is dropped, factors and gradient are exactly zero
    g = run_gpu_layer(B, A, torch.zeros_like(D), Q0, r, 2)
    assert not g["P"].any() and not g["Q"].any() and not g["grad"].any() and not g["full"].any()
    o = oracle.rank_dad_layer(A, torch.zeros_like(D), Q0, 2)
    assert not o["grad"].any()
    # (b) all start vectors equal: the block spans one direction; one vector survives, as in the oracle
    Q0same = Q0[:, :1].expand(S, r, h_out).contiguous()
    g, o = check_layer(oracle, B, A, D, Q0same, r, 2, tol, ortho_tol=1e-3)
    for s in range(S):
        assert [bool(np.any(g["Q"][s][j] != 0.0)) for j in range(r)] == [True, False, False, False]
    # (c) every row of the batch the same: A_s^T D_s has rank one, reproduced exactly by the first component
    A1 = A[:, :1].expand(S, N, h_in).contiguous()
    D1 = D[:, :1].expand(S, N, h_out).contiguous()
    g, o = check_layer(oracle, B, A1, D1, Q0, r, 1, tol, ortho_tol=1e-3)
    assert rel(g["grad"], oracle.full_grad(A1, D1)) <= tol


def test_layer_step_replays_from_a_cuda_graph(B):
    """The calls only enqueue work on the caller's stream and keep no host state between calls, so a whole
    compress -> gather -> reconstruct step can be captured once and replayed on new inputs."""
    dev = torch.device("cuda:0")
    S, N, h_in, h_out, r, iters = 4, 512, 256, 384, 16, 2
    A, D = wl.decaying_layer(S, N, h_in, h_out, 71, torch.bfloat16, dev)
    A2, D2 = wl.decaying_layer(S, N, h_in, h_out, 72, torch.bfloat16, dev)
    Q0 = wl.start_block(S, r, h_out, 71, dev)
    plan = B.LayerPlan(A, D, r, iters)
    plan.step(A, D, Q0)                       # warm-up outside capture (module load, attribute opt-ins)
    torch.cuda.synchronize()
    eager1 = plan.grad.clone()
    plan.step(A2, D2, Q0)
    torch.cuda.synchronize()
    eager2 = plan.grad.clone()
    Ain, Din = A.clone(), D.clone()            # static input buffers of the graph
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            plan.step(Ain, Din, Q0, stream=side)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(plan.grad, eager1)
    Ain.copy_(A2)
    Din.copy_(D2)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(plan.grad, eager2)
    B.dad_check(plan.ws)
