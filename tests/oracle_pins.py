"""Pins of the CPU oracle: each function checks the oracle against something the paper or
the mathematics fixes (never against the oracle's own formula retyped) and raises
AssertionError when it does not hold.  ``test_oracle_pins.py`` runs them on the oracle as
committed; ``test_oracle_mutants.py`` runs them on copies with a planted mistake and
expects at least one to fail.
"""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def planted(N, h_in, h_out, sigmas, seed):
    """A (N x h_in) with orthonormal columns-of-A^T structure and D such that the singular
    values of A^T D are exactly `sigmas` (len <= min(N, h_in, h_out)); returns A, D, U, V."""
    rng = _rng(seed)
    k = len(sigmas)
    assert k <= min(N, h_in, h_out)
    # A^T D = (A^T X) diag(s) V^T with A^T X = U orthonormal: take A = X U^T, X orthonormal N x k.
    X = np.linalg.qr(rng.standard_normal((N, k)))[0]
    U = np.linalg.qr(rng.standard_normal((h_in, k)))[0]
    V = np.linalg.qr(rng.standard_normal((h_out, k)))[0]
    A = X @ U.T
    D = X @ np.diag(sigmas) @ V.T
    return A, D, U, V


def sin_angles(Qa, Qb):
    """Sines of the principal angles between the row spaces of two row-orthonormal matrices."""
    return np.linalg.svd(Qa - (Qa @ Qb.T) @ Qb, compute_uv=False)  # residual of Qa outside span(Qb)


# --------------------------------------------------------------------------- O-1 full_grad
def pin_full_grad_is_pooled_product(o):
    """Sec. 3.2 / 5.1: concatenating all sites on the batch dimension and multiplying gives the
    same matrix (library matmul on the pooled batch)."""
    rng = _rng(1)
    S, N, h_in, h_out = 3, 7, 11, 5
    A = rng.standard_normal((S, N, h_in))
    D = rng.standard_normal((S, N, h_out))
    G = o.full_grad(A, D)
    pooled = A.reshape(S * N, h_in).T @ D.reshape(S * N, h_out)
    assert G.shape == (h_in, h_out)
    assert np.abs(G - pooled).max() <= 1e-12 * np.abs(pooled).max()
    # not symmetric in its arguments: swapping gives the transpose
    assert np.abs(o.full_grad(D, A) - pooled.T).max() <= 1e-12 * np.abs(pooled).max()


def pin_full_grad_is_autograd_gradient(o):
    """Eq. "local_grad" + Sec. 5.1: on the MLP workload, sum_s A_s^T D_s equals the gradient of the
    pooled loss that reverse-mode autodiff (library routine) and central differences give."""
    import torch
    from paper_2102_09631_b200 import workloads as wl

    mb = wl.mlp_layers(S=2, N=6, sizes=(9, 12, 8, 4), seed=77)
    S, N = mb.X.shape[:2]
    W = [w.clone().requires_grad_(True) for w in mb.W]

    def pooled_loss(Ws):
        x = mb.X.reshape(S * N, -1)
        for i, w in enumerate(Ws):
            x = x @ w + mb.b[i]
            if i < len(Ws) - 1:
                x = torch.relu(x)
        return torch.nn.functional.cross_entropy(x, mb.labels.reshape(-1), reduction="mean")

    loss = pooled_loss(W)
    assert abs(float(loss.detach()) - mb.loss) < 1e-12
    loss.backward()
    for i in range(len(W)):
        G = o.full_grad(mb.A[i].numpy(), mb.D[i].numpy())
        ref = W[i].grad.numpy()
        assert np.abs(G - ref).max() <= 1e-12 * max(1.0, np.abs(ref).max()), i
    # central finite differences on a few weights of the middle layer
    G1 = o.full_grad(mb.A[1].numpy(), mb.D[1].numpy())
    eps = 1e-6
    for (a, b) in [(0, 0), (3, 5), (11, 7)]:
        Wp = [w.detach().clone() for w in mb.W]
        Wm = [w.detach().clone() for w in mb.W]
        Wp[1][a, b] += eps
        Wm[1][a, b] -= eps
        fd = (float(pooled_loss(Wp)) - float(pooled_loss(Wm))) / (2 * eps)
        assert abs(fd - G1[a, b]) <= 1e-7, (a, b, fd, G1[a, b])


# --------------------------------------------------------------------------- O-2 reconstruct
def pin_reconstruct_is_sum_of_outer_products(o):
    """Algorithm 1 (P^T Q step): the estimate is the sum over sites and components of outer products."""
    rng = _rng(2)
    S, r, h_in, h_out = 3, 2, 6, 4
    P = rng.standard_normal((S, r, h_in))
    Q = rng.standard_normal((S, r, h_out))
    Pcat, Qcat, tx = o.gather(P, Q)
    G = o.reconstruct(Pcat, Qcat)
    ref = np.zeros((h_in, h_out))
    for s in range(S):
        for j in range(r):
            ref += np.outer(P[s, j], Q[s, j])
    assert np.abs(G - ref).max() < 1e-13
    # same contraction as the uncompressed product with the stacks in the place of (A, D)
    assert np.abs(G - o.full_grad(Pcat[None], Qcat[None])).max() < 1e-13


def pin_gather_stacks_sites_in_order(o):
    """Algorithm 1 (vertcat at the aggregator): site s lands in rows s*r .. s*r+r-1; bytes per site."""
    S, r, h_in, h_out = 3, 2, 5, 4
    P = np.arange(S * r * h_in, dtype=np.float64).reshape(S, r, h_in)
    Q = -np.arange(S * r * h_out, dtype=np.float64).reshape(S, r, h_out)
    Pcat, Qcat, tx = o.gather(P, Q)
    assert Pcat.shape == (S * r, h_in) and Qcat.shape == (S * r, h_out)
    assert np.array_equal(Pcat, np.vstack([P[s] for s in range(S)]))
    assert np.array_equal(Qcat, np.vstack([Q[s] for s in range(S)]))
    assert tx.dtype == np.uint64 and list(tx) == [r * (h_in + h_out) * 4] * S


# --------------------------------------------------------------------------- orth
def pin_orth_is_thin_qr(o):
    """orth = thin QR with positive diagonal: matches the library QR after fixing signs."""
    rng = _rng(3)
    r, h = 5, 17
    G = rng.standard_normal((r, h))
    Q, R = o.orth(G)
    q_np, r_np = np.linalg.qr(G.T)
    sgn = np.sign(np.diag(r_np))
    assert np.abs(Q - (q_np * sgn).T).max() < 1e-12
    assert np.abs(R - np.abs(np.diag(r_np))).max() < 1e-12
    assert (R > 0).all()
    assert np.abs(Q @ Q.T - np.eye(r)).max() < 1e-14


def pin_orth_zeroes_dependent_rows(o):
    """A row inside the span of the earlier rows carries no new direction: exactly zero."""
    rng = _rng(4)
    G = rng.standard_normal((4, 9))
    G[2] = 2.0 * G[0] - 3.0 * G[1]
    Q, R = o.orth(G)
    assert np.all(Q[2] == 0.0) and R[2] == 0.0
    keep = [0, 1, 3]
    assert np.abs(Q[keep] @ Q[keep].T - np.eye(3)).max() < 1e-13
    # the kept rows still span the input's row space
    resid = G - (G @ Q.T) @ Q
    assert np.abs(resid).max() < 1e-12
    Qz, Rz = o.orth(np.zeros((2, 5)))
    assert np.all(Qz == 0.0) and np.all(Rz == 0.0)


# --------------------------------------------------------------------------- O-3 spi_block
def pin_spi_exact_when_rank_fits(o):
    """Sec. 3.3.1 (the true rank can be below r): with r >= rank(A^T D) one application of M already
    spans the row space, and P^T Q reproduces A^T D; the surplus rows of Q are exactly zero."""
    rng = _rng(5)
    # (a) batch smaller than r
    N, h_in, h_out, r = 3, 12, 10, 5
    A = rng.standard_normal((N, h_in))
    D = rng.standard_normal((N, h_out))
    Q0 = rng.standard_normal((r, h_out))
    P, Q, sig = o.spi_block(A, D, Q0, 1)
    gw = A.T @ D
    assert np.linalg.norm(P.T @ Q - gw) <= 1e-10 * np.linalg.norm(gw)
    assert sum(bool(np.all(Q[j] == 0.0)) for j in range(r)) == r - N
    assert np.all(sig[N:] == 0.0)
    # (b) planted rank 3 inside a larger batch, several sites at once
    S, N, r = 2, 20, 4
    A = rng.standard_normal((S, N, h_in))
    D = np.stack([rng.standard_normal((N, 3)) @ rng.standard_normal((3, h_out)) for _ in range(S)])
    Q0 = rng.standard_normal((S, r, h_out))
    P, Q, sig = o.spi_block(A, D, Q0, 1)
    for s in range(S):
        gw = A[s].T @ D[s]
        assert np.linalg.norm(P[s].T @ Q[s] - gw) <= 1e-10 * np.linalg.norm(gw)
    # and the whole per-layer path then equals the uncompressed dAD gradient
    out = o.rank_dad_layer(A, D, Q0, 1)
    full = o.full_grad(A, D)
    assert np.linalg.norm(out["grad"] - full) <= 1e-10 * np.linalg.norm(full)


def pin_spi_finds_svd_subspace(o):
    """Sec. 3.3.1: iterating M converges to the dominant right singular vectors; the textbook rate of
    subspace iteration on M = gradW^T gradW is (sigma_{r+1}/sigma_r)^(2 iters)."""
    sig = np.array([10.0, 8.0, 6.0, 4.0, 1.0, 0.5, 0.25])
    A, D, U, V = planted(12, 15, 13, sig, seed=6)
    r = 4
    Q0 = _rng(60).standard_normal((r, 13))
    gw = A.T @ D
    _, s_np, vt = np.linalg.svd(gw)
    assert np.allclose(s_np[:7], sig)
    prev = None
    for iters in (1, 2, 4, 20):
        P, Q, sg = o.spi_block(A, D, Q0, iters)
        s = sin_angles(Q, vt[:r]).max()
        if prev is not None:
            assert s < prev
        prev = s
        t0 = np.tan(np.arcsin(min(1.0, sin_angles(o.orth(Q0)[0], vt[:r]).max())))
        assert s <= (sig[r] / sig[r - 1]) ** (2 * iters) * t0 * 1.0000001 + 1e-12
    assert prev < 1e-8
    # individual vectors settle at the slower rate (sigma_{j+1}/sigma_j)^2 per application: iterate on
    P, Q, sg = o.spi_block(A, D, Q0, 200)
    # at convergence: sigma = singular values, rows of Q = right vectors, P_j/sigma_j = left vectors
    assert np.allclose(sg, sig[:r], rtol=1e-9)
    for j in range(r):
        assert abs(abs(Q[j] @ vt[j]) - 1.0) < 1e-9
        u = np.linalg.svd(gw)[0][:, j]
        assert abs(abs((P[j] / sg[j]) @ u) - 1.0) < 1e-9
        # sign: P_j, Q_j pair reproduces +sigma_j u_j v_j^T
        assert np.linalg.norm(np.outer(P[j], Q[j]) - sig[j] * np.outer(u, vt[j]) * np.sign((P[j] @ u) * (Q[j] @ vt[j]))) < 1e-7


def pin_spi_invariants(o):
    """What holds for any finite iteration count: Q Q^T = I; P = (gradW Q^T)^T; Pythagoras
    ||gradW - P^T Q||^2 = ||gradW||^2 - ||P||^2; the Eckart-Young lower bound (the factors are the
    least-squares optimal low-rank representation only in the limit); sigma = ||P_j||."""
    rng = _rng(7)
    N, h_in, h_out, r = 14, 9, 11, 3
    A = rng.standard_normal((N, h_in))
    D = rng.standard_normal((N, h_out)) * (1.0 / np.arange(1, h_out + 1))
    Q0 = rng.standard_normal((r, h_out))
    gw = A.T @ D
    sv = np.linalg.svd(gw, compute_uv=False)
    tail = np.sum(sv[r:] ** 2)
    last = None
    for iters in (1, 2, 3, 8, 60):
        P, Q, sg = o.spi_block(A, D, Q0, iters)
        assert np.abs(Q @ Q.T - np.eye(r)).max() < 1e-12
        assert np.abs(P - (gw @ Q.T).T).max() < 1e-12 * np.abs(gw).max() * h_out
        err2 = np.linalg.norm(gw - P.T @ Q) ** 2
        assert abs(err2 - (np.linalg.norm(gw) ** 2 - np.linalg.norm(P) ** 2)) < 1e-10 * np.linalg.norm(gw) ** 2
        assert err2 >= tail * (1 - 1e-10)
        assert np.allclose(sg, np.linalg.norm(P, axis=1), rtol=1e-13)
        if last is not None:
            assert err2 <= last * (1 + 1e-9)
        last = err2
    assert abs(last - tail) < 1e-6 * tail


def pin_spi_span_is_krylov_block(o):
    """Eq. "nabla_iter": after k applications the rows of Q span M^k Q0^T, M built explicitly."""
    rng = _rng(8)
    N, h_in, h_out, r = 10, 8, 7, 3
    A = rng.standard_normal((N, h_in))
    D = rng.standard_normal((N, h_out))
    Q0 = rng.standard_normal((r, h_out))
    gw = A.T @ D
    M = gw.T @ gw
    for iters in (1, 2, 3):
        P, Q, _ = o.spi_block(A, D, Q0, iters)
        K = np.linalg.matrix_power(M, iters) @ Q0.T
        Kq = np.linalg.qr(K)[0]
        assert np.abs(Kq @ Kq.T - Q.T @ Q).max() < 1e-9, iters
        # thin QR with positive diagonal is unique: the rows themselves agree, not only the span
        qk, rk = np.linalg.qr(K)
        assert np.abs((qk * np.sign(np.diag(rk))).T - Q).max() < 1e-8
    # zero iterations: Q is the start block itself and P = (gradW Q0^T)^T
    P, Q, _ = o.spi_block(A, D, Q0, 0)
    assert np.array_equal(Q, Q0) and np.abs(P - (gw @ Q0.T).T).max() < 1e-12


def pin_paper_identities(o):
    """Sec. 3.3.1: with C = A A^T and B = D^T C, B D = gradW^T gradW (Eq. "reduced_iter"), and
    sigma = sqrt(v^T C v) with v = D g equals ||A^T v|| -- the sigma the oracle reports."""
    rng = _rng(9)
    N, h_in, h_out = 6, 9, 8
    A = rng.standard_normal((N, h_in))
    D = rng.standard_normal((N, h_out))
    C = A @ A.T
    B = D.T @ C
    gw = A.T @ D
    assert np.abs(B @ D - gw.T @ gw).max() < 1e-11
    Q0 = rng.standard_normal((2, h_out))
    P, Q, sg = o.spi_block(A, D, Q0, 2)
    for j in range(2):
        v = D @ Q[j]
        assert abs(np.sqrt(v @ C @ v) - sg[j]) < 1e-11 * sg[j]
        assert np.abs(A.T @ v - P[j]).max() < 1e-12
    # one iteration from a single start vector is B (D g) normalised
    P1, Q1, _ = o.spi_block(A, D, Q0[:1], 1)
    g = B @ (D @ Q0[0])
    assert np.abs(Q1[0] - g / np.linalg.norm(g)).max() < 1e-12


def pin_sites_are_independent(o):
    """Algorithm 1: SPI runs per site; the S-site call equals S single-site calls."""
    rng = _rng(10)
    S, N, h_in, h_out, r = 3, 8, 6, 7, 2
    A = rng.standard_normal((S, N, h_in))
    D = rng.standard_normal((S, N, h_out))
    Q0 = rng.standard_normal((S, r, h_out))
    P, Q, sg = o.spi_block(A, D, Q0, 2)
    for s in range(S):
        Ps, Qs, ss = o.spi_block(A[s], D[s], Q0[s], 2)
        assert np.array_equal(P[s], Ps) and np.array_equal(Q[s], Qs) and np.array_equal(sg[s], ss)


# --------------------------------------------------------------------------- O-4 spi_paper
def pin_spi_paper_first_vector_is_power_iteration(o):
    """Eq. "nabla_iter": for the first component Algorithm 2 is plain power iteration on the explicit M."""
    rng = _rng(11)
    N, h_in, h_out = 9, 7, 6
    A = rng.standard_normal((N, h_in))
    D = rng.standard_normal((N, h_out))
    g0 = rng.standard_normal((1, h_out))
    M = (A.T @ D).T @ (A.T @ D)
    g = g0[0] / np.linalg.norm(g0[0])
    for _ in range(5):
        g = M @ g
        g /= np.linalg.norm(g)
    P, Q, sg = o.spi_paper(A, D, g0, 5)
    assert np.abs(Q[0] - g).max() < 1e-12
    assert np.abs(P[0] - A.T @ (D @ g)).max() < 1e-12
    assert abs(sg[0] - np.linalg.norm(A.T @ D @ g)) < 1e-12


def pin_spi_paper_matches_block_form(o):
    """The sequential (peeled) and the blocked form find the same subspace: both reach the SVD's
    when iterated to convergence, and both are exact once r >= rank."""
    sig = np.array([9.0, 7.0, 5.0, 1.0, 0.5])
    A, D, U, V = planted(10, 12, 11, sig, seed=12)
    r = 3
    Q0 = _rng(120).standard_normal((r, 11))
    Pb, Qb, sb = o.spi_block(A, D, Q0, 25)
    Pp, Qp, sp = o.spi_paper(A, D, Q0, 60)
    assert sin_angles(Qb, Qp).max() < 1e-8
    assert np.allclose(sp, sig[:r], rtol=1e-8) and np.allclose(sb, sig[:r], rtol=1e-8)
    assert np.abs(Qp @ Qp.T - np.eye(r)).max() < 1e-12
    gw = A.T @ D
    assert np.linalg.norm(Pp.T @ Qp - Pb.T @ Qb) < 1e-7 * np.linalg.norm(gw)
    # exactness with r >= rank
    rng = _rng(13)
    A = rng.standard_normal((3, 8))
    D = rng.standard_normal((3, 9))
    Q0 = rng.standard_normal((4, 9))
    Pp, Qp, sp = o.spi_paper(A, D, Q0, 40)
    gw = A.T @ D
    assert np.linalg.norm(Pp.T @ Qp - gw) < 1e-8 * np.linalg.norm(gw)
    assert np.all(Qp[3] == 0.0)


# --------------------------------------------------------------------------- O-5 bytes
def read_golden_bytes():
    rows = []
    with open(os.path.join(GOLDEN, "bytes_per_site.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                rows.append([int(x) for x in line.split()])
    return rows


def pin_bytes_closed_forms(o):
    """Sec. 3.1 (m+n against m*n per sample), Sec. 3.2 (N(h_in+h_out) against h_in*h_out), Sec. 2
    (Theta(r(h_i+h_{i+1})) for rank methods): tabulated values worked out by hand."""
    for N, h_in, h_out, e, r, dsgd, dad, rank in read_golden_bytes():
        assert o.bytes_dsgd(h_in, h_out) == dsgd
        assert o.bytes_dad(N, h_in, h_out, e) == dad
        assert o.bytes_rank(r, h_in, h_out) == rank
    # one sample, fp32: m+n values against m*n
    assert o.bytes_dad(1, 300, 500, 4) == 4 * (300 + 500) and o.bytes_dsgd(300, 500) == 4 * 300 * 500
    # linear in r and in (h_in + h_out)
    assert o.bytes_rank(6, 10, 20) == 2 * o.bytes_rank(3, 10, 20) == o.bytes_rank(3, 20, 40)
    # crossover (Sec. 3.2): dAD saves only when N(h_in+h_out)e < 4 h_in h_out
    assert o.bytes_dad(128, 1024, 10, 4) > o.bytes_dsgd(1024, 10)
    assert o.bytes_dad(128, 1024, 1024, 4) < o.bytes_dsgd(1024, 1024)
    # no 32-bit wrap
    assert o.bytes_dad(1 << 20, 1 << 14, 1 << 14, 4) == (1 << 20) * (1 << 15) * 4


# --------------------------------------------------------------------------- aggregator SPI, effective rank
def pin_two_stage_is_spi_of_the_stacks(o):
    """Algorithm 1 (SPI at the aggregator): Phat^T Qhat is the projection of Pcat^T Qcat = sum_s P_s^T Q_s on
    r directions; exact once r covers the rank of the stacked product, never better than Eckart-Young, and the
    optimum in the limit."""
    rng = _rng(21)
    S, N, h_in, h_out, r = 3, 9, 10, 8, 2
    A = rng.standard_normal((S, N, h_in))
    D = rng.standard_normal((S, N, h_out)) * (1.0 / np.arange(1, h_out + 1))
    Q0 = rng.standard_normal((S, r, h_out))
    # aggregator rank 6 = S * r >= rank of the stacked product: nothing is lost
    out = o.two_stage_layer(A, D, Q0, 2, rng.standard_normal((S * r, h_out)), 1)
    assert np.linalg.norm(out["grad_hat"] - out["grad"]) <= 1e-10 * np.linalg.norm(out["grad"])
    # aggregator rank 2 < 6: a rank-2 projection of the stacked product
    Q0a = rng.standard_normal((2, h_out))
    target = out["grad"]
    sv = np.linalg.svd(target, compute_uv=False)
    last = None
    for it in (1, 3, 40):
        o2 = o.two_stage_layer(A, D, Q0, 2, Q0a, it)
        Ph, Qh = o2["Phat"], o2["Qhat"]
        assert np.abs(Qh @ Qh.T - np.eye(2)).max() < 1e-12
        assert np.abs(Ph - (target @ Qh.T).T).max() < 1e-11 * np.abs(target).max() * h_out
        err2 = np.linalg.norm(target - o2["grad_hat"]) ** 2
        assert err2 >= np.sum(sv[2:] ** 2) * (1 - 1e-10)
        if last is not None:
            assert err2 <= last * (1 + 1e-9)
        last = err2
        assert o2["bytes_down"] == 2 * (h_in + h_out) * 4 and list(o2["bytes_tx"]) == [r * (h_in + h_out) * 4] * S
    assert abs(last - np.sum(sv[2:] ** 2)) < 1e-8 * np.sum(sv ** 2)


def pin_effective_rank_worked_cases(o):
    """Sec. 3.3.1 / Algorithm 2 early stop, theta = 1e-3: hand-worked cases of the rule that is implemented."""
    with open(os.path.join(GOLDEN, "effective_rank.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            theta, sig, want = [x.strip() for x in line.split("|")]
            got = o.effective_rank(np.array([float(x) for x in sig.split()], dtype=np.float32), float(theta))
            assert list(got) == [int(want)], (line, got)
    # several sites at once are handled independently; truncation zeroes exactly the dropped components
    sg = np.array([[4, 2, 1e-4, 1], [1, 0.5, 0.25, 0.125]], dtype=np.float32)
    k = o.effective_rank(sg, 1e-3)
    assert list(k) == [2, 4]
    P = np.ones((2, 4, 3))
    Q = np.ones((2, 4, 5))
    Pt, Qt = o.truncate(P, Q, k)
    assert Pt[0, 2:].sum() == 0 and Qt[0, 2:].sum() == 0 and Pt[0, :2].sum() == 6 and Pt[1].sum() == 12
    # dropping a noise component changes the estimate by no more than its strength
    rng = _rng(22)
    A, D, U, V = planted(12, 9, 10, np.array([5.0, 3.0, 1e-5]), seed=23)
    Pf, Qf, sf = o.spi_block(A, D, rng.standard_normal((3, 10)), 30)
    keep = o.effective_rank(sf.astype(np.float32), 1e-3)
    assert list(keep) == [2]
    Pt, Qt = o.truncate(Pf[None], Qf[None], keep)
    assert np.linalg.norm(Pt[0].T @ Qt[0] - Pf.T @ Qf) <= 1.0001e-5


def pin_spi_gram_form_equals_structured_form(o):
    """Sec. 3.3.1, Eq. "reduced_iter": iterating B (D g) with B = D^T C, C = A A^T is the same recurrence as
    gradW^T gradW g, so Algorithm 2 with its precomputed matrices gives the factors of the right-to-left form;
    and its sigma = sqrt(v^T C v) is the singular value at convergence."""
    rng = _rng(31)
    S, N, h_in, h_out, r = 2, 6, 14, 11, 3
    A = rng.standard_normal((S, N, h_in))
    D = rng.standard_normal((S, N, h_out))
    Q0 = rng.standard_normal((S, r, h_out))
    for iters in (0, 1, 3):
        Pg, Qg, sg = o.spi_gram(A, D, Q0, iters)
        Pb, Qb, sb = o.spi_block(A, D, Q0, iters)
        assert np.abs(Pg - Pb).max() < 1e-9 and np.abs(Qg - Qb).max() < 1e-9 and np.abs(sg - sb).max() < 1e-9
    # against the explicit operator, one step from one vector
    gw = A[0].T @ D[0]
    P1, Q1, s1 = o.spi_gram(A[0], D[0], Q0[0, :1], 1)
    g = gw.T @ (gw @ Q0[0, 0])
    g /= np.linalg.norm(g)
    assert np.abs(Q1[0] - g).max() < 1e-12 and abs(s1[0] - np.linalg.norm(gw @ g)) < 1e-11
    # converged: sigma are the singular values
    sig = np.array([6.0, 3.0, 1.0])
    Ap, Dp, U, V = planted(8, 10, 9, sig, seed=32)
    Pc, Qc, sc = o.spi_gram(Ap, Dp, rng.standard_normal((3, 9)), 80)
    assert np.allclose(sc, sig, rtol=1e-9)


ALL_PINS = [v for k, v in sorted(globals().items()) if k.startswith("pin_") and callable(v)]
