"""Pins of the CPU oracle against things other than itself: published test vectors, library
routines (numpy.linalg, torch.optim), closed forms, invariants the paper states, brute force."""
import math

import numpy as np
import pytest
import torch

from oracle import lordo_oracle as lo
from oracle.lordo_oracle import (GLOBAL, LOCAL, OUTER_AVG, OUTER_NESTEROV, QHM_FULL, QHM_LOW, QHM_NONE, LordoOracle,
                                 OracleConfig)

RNG = np.random.default_rng(1234)


def subspace_angle(A, B):
    """Largest principal angle between the column spans of two orthonormal bases."""
    s = np.linalg.svd(A.T @ B, compute_uv=False)
    return float(np.arccos(np.clip(s.min(), -1.0, 1.0)))


def make(mats, K=1, H=1, **kw):
    kw.setdefault("state_dtype", "f64")
    kw.setdefault("w_dtype", "f64")
    kw.setdefault("e_dtype", "f64")
    cfg = OracleConfig(mats=tuple(mats), K=K, H=H, **kw)
    W0 = [RNG.standard_normal((m, n)) * 0.02 for m, n, _ in mats]
    return cfg, W0


# ------------------------------------------------------------------ integer generator (R14)

def test_splitmix64_published_vectors():
    # first three outputs of the public-domain splitmix64 generator seeded with 0
    want = [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    got = lo.random_words(0, 3)
    assert [int(x) for x in got] == want
    assert [lo.mix64_int(lo._GOLDEN * (i + 1)) for i in range(3)] == want


def test_vector_and_scalar_generators_agree_and_popcount():
    key = lo.stream_key(7, lo.PURPOSE_OMEGA, 3, 2, 1)
    w = lo.random_words(key, 1000)
    for c in (0, 1, 17, 999):
        assert int(w[c]) == lo.mix64_int(key + lo._GOLDEN * (c + 1))
    pc = lo.popcount64(w)
    assert [bin(int(x)).count("1") for x in w[:200]] == list(pc[:200])
    # distinct streams differ
    assert lo.stream_key(7, 2, 3, 2, 1) != lo.stream_key(7, 2, 3, 2, 0) != lo.stream_key(7, 2, 3, 1, 1)


def test_random_matrix_moments():
    M = lo.random_matrix(0, lo.PURPOSE_OMEGA, 0, 0, 0, 400, 256)
    assert M.shape == (400, 256) and np.all(M == np.round(M)) and np.abs(M).max() <= 32
    assert abs(M.mean()) < 0.05 and abs(M.var() - 16.0) < 0.3  # Binomial(64,1/2): variance 16
    # row-major counter: element (i, j) is word i*cols + j
    w = lo.random_words(lo.stream_key(0, lo.PURPOSE_OMEGA, 0, 0, 0), 400 * 256)
    assert M[3, 5] == bin(int(w[3 * 256 + 5])).count("1") - 32


def test_round_bf16_matches_torch():
    x = np.concatenate([RNG.standard_normal(5000) * 10.0 ** RNG.integers(-6, 6, 5000),
                        np.array([1.00390625, 1.01171875, -1.00390625, 0.0, 65280.0, 1e-40])])
    want = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(lo.round_bf16(x), want)


# ------------------------------------------------------------------ QR and the range finder (R1)

@pytest.mark.parametrize("rows,r", [(8, 8), (50, 7), (300, 64)])
def test_householder_matches_numpy_qr(rows, r):
    Y = RNG.standard_normal((rows, r))
    Q = lo.householder_qr_q(Y)
    q, rr = np.linalg.qr(Y)
    q = q * np.sign(np.diag(rr))[None, :]
    assert np.abs(Q - q).max() < 1e-10
    assert np.abs(Q.T @ Q - np.eye(r)).max() < 1e-12
    R = Q.T @ Y
    assert np.all(np.diag(R) > 0) and np.abs(np.tril(R, -1)).max() < 1e-10


def test_householder_rank_deficient_is_finite_and_orthonormal():
    Y = RNG.standard_normal((40, 3)) @ RNG.standard_normal((3, 8))
    Y[:, 5] = 0.0
    Q = lo.householder_qr_q(Y)
    assert np.all(np.isfinite(Q)) and np.abs(Q.T @ Q - np.eye(8)).max() < 1e-10


def test_initial_projection_orthonormal():
    cfg, W0 = make([(96, 40, 16), (64, 64, 8)], K=2)
    o = LordoOracle(cfg, W0)
    for P in o.P:
        assert np.abs(P.T @ P - np.eye(P.shape[1])).max() < 1e-5
    cfgl, _ = make([(96, 40, 16)], K=2, variant=LOCAL)
    ol = LordoOracle(cfgl, W0[:1])
    assert ol.P[0].shape == (2, 96, 16) and np.array_equal(ol.P[0][1], np.eye(96, 16))


@pytest.mark.parametrize("q", [0, 2])
def test_exact_low_rank_gradient_is_reconstructed(q):
    m, n, r = 64, 48, 8
    cfg, W0 = make([(m, n, r)], K=1, variant=LOCAL, power_iters=q)
    o = LordoOracle(cfg, W0)
    G = [(RNG.standard_normal((m, r)) @ RNG.standard_normal((r, n)))[None]]
    o.refresh_subspace(G)
    P = o.P[0][0]
    assert np.abs(P.T @ P - np.eye(r)).max() < 1e-5
    assert np.linalg.norm(G[0][0] - P @ (P.T @ G[0][0])) / np.linalg.norm(G[0][0]) < 1e-5
    o.inner_step(G, 1e-3, 0.9, 1.0, QHM_NONE)
    assert np.abs(o.E[0]).max() < 1e-10 * np.abs(G[0]).max()


@pytest.mark.parametrize("q", [0, 1, 2])
def test_range_finder_angle_equals_closed_form(q):
    """For S = U diag(s) V^T the span of (S S^T)^q S Omega is the span of U [I ; T] with
    T = S2^(2q+1) Om2 Om1^-1 S1^-(2q+1), Om1 = V1^T Omega, Om2 = V2^T Omega, so the largest
    principal angle to the top-r singular subspace (the paper's target, Q = U[:, :r]) has
    tan(theta) = ||T||_2 exactly. It decays like (s_{r+1}/s_r)^(2q+1)."""
    m, n, r = 80, 60, 6
    U, _ = np.linalg.qr(RNG.standard_normal((m, m)))
    V, _ = np.linalg.qr(RNG.standard_normal((n, n)))
    sv = np.concatenate([np.linspace(10, 5, r), np.linspace(0.5, 0.05, n - r)])
    S = (U[:, :n] * sv) @ V.T
    Om = lo.random_matrix(0, lo.PURPOSE_OMEGA, 0, 0, 0, n, r)
    P = lo.compute_projection(S, Om, q)
    Om1, Om2 = V[:, :r].T @ Om, V[:, r:].T @ Om
    e = 2 * q + 1
    T = (sv[r:, None] ** e) * (Om2 @ np.linalg.inv(Om1)) / (sv[None, :r] ** e)
    want = math.atan(np.linalg.norm(T, 2))
    got = subspace_angle(P, U[:, :r])
    assert abs(got - want) < 1e-6 * max(want, 1e-3) + 1e-9
    Sx = (U[:, :r] * sv[:r]) @ V[:, :r].T  # exact rank r: the subspace is recovered exactly
    assert subspace_angle(lo.compute_projection(Sx, Om, q), U[:, :r]) < 1e-6


# ------------------------------------------------------------------ reductions to Adam

def _adam_reference(W0, grads, lr, b1, b2, eps):
    w = torch.tensor(W0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([w], lr=lr, betas=(b1, b2), eps=eps, weight_decay=0.0)
    for g in grads:
        w.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
    return w.detach().numpy()


def test_identity_projection_reduces_to_adam():
    m, n = 8, 12
    cfg, W0 = make([(m, n, m)], K=1, H=1, variant=LOCAL, eps=1e-8, beta2=0.999)
    o = LordoOracle(cfg, W0)  # Local: Q_0 = I
    grads = [RNG.standard_normal((m, n)) for _ in range(6)]
    for g in grads:
        o.inner_step([g[None]], 3e-3, 0.9, 1.0, QHM_NONE)
        o.outer_step()  # K = 1, averaging: must be the identity
    want = _adam_reference(W0[0], grads, 3e-3, 0.9, 0.999, 1e-8)
    assert np.abs(o.W[0][0] - want).max() < 1e-13
    assert np.abs(o.E[0]).max() == 0.0


def test_square_orthogonal_projection_is_adam_in_rotated_coordinates():
    m, n = 10, 7
    Qo, _ = np.linalg.qr(RNG.standard_normal((m, m)))
    cfg, W0 = make([(m, n, m)], K=1, H=1)
    o = LordoOracle(cfg, W0, P0=[Qo])
    grads = [RNG.standard_normal((m, n)) for _ in range(5)]
    for g in grads:
        o.inner_step([g[None]], 1e-2, 0.8, 1.0, QHM_NONE)
    want = Qo @ _adam_reference(Qo.T @ W0[0], [Qo.T @ g for g in grads], 1e-2, 0.8, 0.999, 1e-8)
    assert np.abs(o.W[0][0] - want).max() < 1e-12


# ------------------------------------------------------------------ brute force on 8x8

def _brute_inner(W, E, P, u, v, G, s, lr, b1, b2, eps, omega, form, rho, ef):
    """Direct loops over Algorithm 1's per-step lines for one worker; python floats only."""
    m, n, r = len(W), len(W[0]), len(P[0])
    nrm = math.sqrt(sum(G[i][j] ** 2 for i in range(m) for j in range(n)))
    c = min(1.0, rho / (nrm + 1e-6)) if rho > 0 else 1.0
    A = [[c * G[i][j] + (E[i][j] if ef else 0.0) for j in range(n)] for i in range(m)]
    g = [[sum(P[i][a] * A[i][j] for i in range(m)) for j in range(n)] for a in range(r)]
    En = [[A[i][j] - sum(P[i][a] * g[a][j] for a in range(r)) for j in range(n)] for i in range(m)] if ef else E
    un = [[b1 * u[a][j] + (1 - b1) * g[a][j] for j in range(n)] for a in range(r)]
    vn = [[b2 * v[a][j] + (1 - b2) * g[a][j] ** 2 for j in range(n)] for a in range(r)]
    D = [[math.sqrt(vn[a][j] / (1 - b2 ** s)) + eps for j in range(n)] for a in range(r)]
    uh = [[un[a][j] / (1 - b1 ** s) for j in range(n)] for a in range(r)]
    Wn = [[0.0] * n for _ in range(m)]
    for i in range(m):
        for j in range(n):
            if form == QHM_NONE:
                upd = sum(P[i][a] * uh[a][j] / D[a][j] for a in range(r))
            elif form == QHM_LOW:
                upd = sum(P[i][a] * (omega * uh[a][j] + (1 - omega) * g[a][j]) / D[a][j] for a in range(r))
            else:
                mu = sum(D[a][j] for a in range(r)) / r
                upd = (1 - omega) * c * G[i][j] / mu + omega * sum(P[i][a] * uh[a][j] / D[a][j] for a in range(r))
            Wn[i][j] = W[i][j] - lr * upd
    return Wn, En, un, vn


@pytest.mark.parametrize("form", [QHM_NONE, QHM_LOW, QHM_FULL])
@pytest.mark.parametrize("ef", [True, False])
def test_brute_force_8x8_inner_and_outer(form, ef):
    m = n = 8
    r, K, H = 3, 2, 3
    cfg, W0 = make([(m, n, r)], K=K, H=H, clip_rho=2.0, error_feedback=ef, outer=OUTER_NESTEROV, outer_lr=0.7,
                   outer_momentum=0.9, beta2=0.95, eps=1e-6)
    o = LordoOracle(cfg, W0)
    P = o.P[0].tolist()
    W = [W0[0].tolist() for _ in range(K)]
    E = [[[0.0] * n for _ in range(m)] for _ in range(K)]
    u = [[[0.0] * n for _ in range(r)] for _ in range(K)]
    v = [[[0.0] * n for _ in range(r)] for _ in range(K)]
    X0 = W0[0].tolist()
    B = [[0.0] * n for _ in range(m)]
    s = 0
    for rnd in range(2):
        for h in range(H):
            G = RNG.standard_normal((K, m, n)) * (3.0 if h == 1 else 0.1)  # one step clips, others do not
            o.inner_step([G], 0.01, 0.9, 0.7, form)
            s += 1
            for k in range(K):
                W[k], E[k], u[k], v[k] = _brute_inner(W[k], E[k], P, u[k], v[k], G[k].tolist(), s, 0.01, 0.9, 0.95,
                                                      1e-6, 0.7, form, 2.0, ef)
            assert np.abs(o.W[0] - np.array(W)).max() < 1e-13
            assert np.abs(o.E[0] - np.array(E)).max() < 1e-13
            assert np.abs(o.v[0] - np.array(v)).max() < 1e-14
        o.outer_step()
        for a in range(r):
            for j in range(n):
                mu_, mv_ = sum(u[k][a][j] for k in range(K)) / K, sum(v[k][a][j] for k in range(K)) / K
                for k in range(K):
                    u[k][a][j], v[k][a][j] = mu_, mv_
        for i in range(m):
            for j in range(n):
                d = X0[i][j] - sum(W[k][i][j] for k in range(K)) / K
                B[i][j] = 0.9 * B[i][j] + d
                X0[i][j] = X0[i][j] - 0.7 * (d + 0.9 * B[i][j])
                for k in range(K):
                    W[k][i][j] = X0[i][j]
        assert np.abs(o.W[0] - np.array(W)).max() < 1e-13
        assert np.abs(o.u[0] - np.array(u)).max() < 1e-14
        assert np.abs(o.B[0] - np.array(B)).max() < 1e-13


def test_brute_force_8x8_subspace_vs_svd():
    m = n = 8
    r = 2
    U, _ = np.linalg.qr(RNG.standard_normal((m, m)))
    V, _ = np.linalg.qr(RNG.standard_normal((n, n)))
    S = (U * np.array([9, 7, 1e-3, 1e-3, 1e-3, 1e-3, 1e-3, 1e-3])) @ V.T
    Usvd = np.linalg.svd(S)[0][:, :r]  # the paper's definition: Q = U[:, :r]
    P = lo.compute_projection(S, lo.random_matrix(3, lo.PURPOSE_OMEGA, 0, 0, 0, n, r), 1)
    assert subspace_angle(P, Usvd) < 1e-6


def test_brute_force_rotation_8x8():
    r, n, m = 3, 8, 8
    P_old, _ = np.linalg.qr(RNG.standard_normal((m, r)))
    P_new, _ = np.linalg.qr(RNG.standard_normal((m, r)))
    u, v = RNG.standard_normal((r, n)), RNG.random((r, n))
    b1, b2, s = 0.9, 0.99, 5
    un, vn = lo.rotate_moments(u, v, P_new, P_old, b1, b2, s)
    for a in range(r):
        for j in range(n):
            acc_u = acc_v = acc_ru = 0.0
            for b in range(r):
                rot = sum(P_new[i, a] * P_old[i, b] for i in range(m))
                uh, vh = u[b, j] / (1 - b1 ** s), v[b, j] / (1 - b2 ** s)
                acc_u += rot * u[b, j]
                acc_ru += rot * uh
                acc_v += rot * rot * (vh - uh * uh)
            assert abs(un[a, j] - acc_u) < 1e-13
            assert abs(vn[a, j] - (1 - b2 ** s) * abs(acc_v + acc_ru ** 2)) < 1e-13


# ------------------------------------------------------------------ moment rotation (R4, R5)

def test_rotation_identity_and_signed_permutation():
    m, n, r = 20, 9, 5
    P, _ = np.linalg.qr(RNG.standard_normal((m, r)))
    u, v = RNG.standard_normal((r, n)), RNG.random((r, n)) + 1.0  # v_hat >= u_hat^2 not required
    un, vn = lo.rotate_moments(u, v, P, P, 0.9, 0.999, 7)
    assert np.abs(un - u).max() < 1e-13 and np.abs(vn - np.abs(v)).max() < 1e-12
    perm = RNG.permutation(r)
    sign = RNG.choice([-1.0, 1.0], r)
    P2 = P[:, perm] * sign[None, :]
    un, vn = lo.rotate_moments(u, v, P2, P, 0.9, 0.999, 7)
    assert np.abs(un - sign[:, None] * u[perm]).max() < 1e-13
    assert np.abs(vn - v[perm]).max() < 1e-12


# ------------------------------------------------------------------ error feedback

def test_error_feedback_invariants():
    m, n, r = 24, 16, 4
    cfg, W0 = make([(m, n, r)], K=1, clip_rho=0.0)
    o = LordoOracle(cfg, W0)
    o2 = LordoOracle(OracleConfig(**{**cfg.__dict__, "error_feedback": False}), W0)
    P = o.P[0]
    for t in range(4):
        G = [RNG.standard_normal((1, m, n))]
        o.inner_step(G, 1e-3, 0.9, 1.0, QHM_NONE)
        o2.inner_step(G, 1e-3, 0.9, 1.0, QHM_NONE)
        assert np.abs(P.T @ o.E[0][0]).max() < 1e-12  # E is orthogonal to the basis
    # hence with a fixed basis the projected signal, and the whole trajectory, equal the one without EF
    assert np.abs(o.W[0] - o2.W[0]).max() < 1e-12
    assert np.abs(o.E[0]).max() > 0.1


# ------------------------------------------------------------------ stagnation of the global rule

@pytest.mark.parametrize("form,stagnates", [(QHM_NONE, True), (QHM_LOW, True), (QHM_FULL, False)])
def test_global_projection_stagnates_without_full_rank_qhm(form, stagnates):
    m, n, r, K, H = 32, 24, 4, 3, 5
    cfg, W0 = make([(m, n, r)], K=K, H=H)
    o = LordoOracle(cfg, W0)
    P_before = o.P[0].copy()
    for h in range(H):
        o.inner_step([RNG.standard_normal((K, m, n))], 1e-2, 0.9, 0.9, form)
    o.outer_step()
    D = o.Delta[0]
    resid = np.linalg.norm(D - P_before @ (P_before.T @ D)) / np.linalg.norm(D)
    if stagnates:
        assert resid < 1e-10 and np.linalg.matrix_rank(D, tol=1e-9) <= r
        o.refresh_subspace(None, 0.9)
        Rot = o.P[0].T @ P_before
        mssv = np.sum(np.linalg.svd(Rot, compute_uv=False) ** 2) / r
        assert subspace_angle(o.P[0], P_before) < 1e-6 and abs(mssv - 1.0) < 1e-9
    else:
        assert resid > 1e-2


def test_local_pseudo_gradient_rank_bound():
    m, n, r, K, H = 40, 36, 3, 4, 3
    cfg, W0 = make([(m, n, r)], K=K, H=H, variant=LOCAL)
    o = LordoOracle(cfg, W0)
    for h in range(H):
        G = [RNG.standard_normal((K, m, n))]
        if h == 0:
            o.refresh_subspace(G, 0.9)
        o.inner_step(G, 1e-2, 0.9, 0.9, QHM_LOW)
    o.outer_step()
    sv = np.linalg.svd(o.Delta[0], compute_uv=False)
    assert np.sum(sv > 1e-9 * sv[0]) == K * r  # rank(Delta) <= M * r, and generically equal


# ------------------------------------------------------------------ outer step (R9, R10)

def test_outer_average_and_unit_nesterov():
    m, n, r, K = 6, 5, 2, 3
    for kw in (dict(outer=OUTER_AVG), dict(outer=OUTER_NESTEROV, outer_lr=1.0, outer_momentum=0.0)):
        cfg, W0 = make([(m, n, r)], K=K, H=1, **kw)
        o = LordoOracle(cfg, W0)
        o.W[0] = RNG.standard_normal((K, m, n))
        mean = o.W[0].mean(axis=0)
        o.outer_step()
        assert np.abs(o.X0[0] - mean).max() < 1e-14 and np.abs(o.W[0] - mean[None]).max() < 1e-14
        assert np.abs(o.Delta[0] - (W0[0] - mean)).max() < 1e-14


def test_outer_nesterov_matches_torch_sgd():
    m, n, r, K = 5, 4, 2, 2
    cfg, W0 = make([(m, n, r)], K=K, H=1, outer=OUTER_NESTEROV, outer_lr=0.6, outer_momentum=0.9)
    o = LordoOracle(cfg, W0)
    w = torch.tensor(W0[0], dtype=torch.float64, requires_grad=True)
    sgd = torch.optim.SGD([w], lr=0.6, momentum=0.9, nesterov=True, dampening=0.0)
    for t in range(5):
        drift = RNG.standard_normal((K, m, n)) * 0.1
        o.W[0] = o.W[0] + drift  # workers move away from the anchor
        delta = -(drift.mean(axis=0))
        w.grad = torch.tensor(delta)
        sgd.step()
        o.outer_step()
        assert np.abs(o.Delta[0] - delta).max() < 1e-14
        assert np.abs(o.X0[0] - w.detach().numpy()).max() < 1e-13
    # constant pseudo-gradient: B_j = Delta (1 - mu^j) / (1 - mu)
    cfg2, W02 = make([(m, n, r)], K=1, H=1, outer=OUTER_NESTEROV, outer_lr=0.5, outer_momentum=0.8)
    o2 = LordoOracle(cfg2, W02)
    d = RNG.standard_normal((m, n))
    for j in range(1, 6):
        o2.W[0] = (o2.X0[0] - d)[None]
        o2.outer_step()
        assert np.abs(o2.B[0] - d * (1 - 0.8 ** j) / (1 - 0.8)).max() < 1e-13


def test_single_worker_means_are_identities_and_state_sync():
    m, n, r = 6, 7, 2
    cfg, W0 = make([(m, n, r)], K=1, H=2)
    o = LordoOracle(cfg, W0)
    for _ in range(2):
        o.inner_step([RNG.standard_normal((1, m, n))], 1e-2, 0.9, 1.0, QHM_NONE)
    u, v, W = o.u[0].copy(), o.v[0].copy(), o.W[0].copy()
    o.outer_step()
    assert np.array_equal(o.u[0], u) and np.array_equal(o.v[0], v) and np.abs(o.W[0] - W).max() < 1e-16
    cfg3, W03 = make([(m, n, r)], K=3, H=1, sync_u=True, sync_v=False)
    o3 = LordoOracle(cfg3, W03)
    o3.inner_step([RNG.standard_normal((3, m, n))], 1e-2, 0.9, 1.0, QHM_NONE)
    u3, v3 = o3.u[0].copy(), o3.v[0].copy()
    o3.outer_step()
    assert np.abs(o3.u[0] - u3.mean(axis=0)[None]).max() < 1e-16 and np.array_equal(o3.v[0], v3)


# ------------------------------------------------------------------ sign invariance

def test_column_sign_flips_leave_weights_unchanged_but_rotations_do_not():
    m, n, r = 16, 12, 4
    cfg, W0 = make([(m, n, r)], K=1)
    P, _ = np.linalg.qr(RNG.standard_normal((m, r)))
    sign = np.array([1.0, -1.0, -1.0, 1.0])
    Rq, _ = np.linalg.qr(RNG.standard_normal((r, r)))
    oa, ob, oc = (LordoOracle(cfg, W0, P0=[p]) for p in (P, P * sign[None], P @ Rq))
    for t in range(3):
        G = [RNG.standard_normal((1, m, n))]
        for o in (oa, ob, oc):
            o.inner_step(G, 1e-2, 0.9, 0.8, QHM_FULL)
    assert np.abs(oa.W[0] - ob.W[0]).max() < 1e-14
    assert np.abs(oa.u[0] - sign[None, :, None] * ob.u[0]).max() < 1e-14
    assert np.abs(oa.W[0] - oc.W[0]).max() > 1e-4


# ------------------------------------------------------------------ clipping (R8)

def test_clip_matches_torch_clip_grad_norm():
    shapes = [(6, 5), (4, 9)]
    K = 3
    G = [RNG.standard_normal((K, a, b)) * sc for (a, b), sc in zip(shapes, (2.0, 0.5))]
    G[0][2] *= 0.01
    G[1][2] *= 0.01  # worker 2 stays under the radius
    rho = 1.5
    coef = lo.clip_coefficients(G, rho, 0)
    for k in range(K):
        params = [torch.nn.Parameter(torch.zeros(a, b, dtype=torch.float64)) for a, b in shapes]
        for p, g in zip(params, G):
            p.grad = torch.tensor(g[k])
        total = torch.nn.utils.clip_grad_norm_(params, rho)
        for i, p in enumerate(params):
            assert np.abs(p.grad.numpy() - coef[i, k] * G[i][k]).max() < 1e-12
        clipped = math.sqrt(sum(np.sum((coef[i, k] * G[i][k]) ** 2) for i in range(2)))
        assert clipped <= rho * (1 + 1e-6)
        assert coef[0, k] == coef[1, k]
    assert coef[0, 2] == 1.0 and coef[0, 0] < 1.0
    per_mat = lo.clip_coefficients(G, rho, 1)
    assert per_mat[0, 0] != per_mat[1, 0]
    assert np.all(lo.clip_coefficients(G, 0.0) == 1.0)


# ------------------------------------------------------------------ storage accounting

def test_state_size_matches_memory_table():
    # Table "Memory overhead": parameters pq + projection pr + states 2rq (+ error buffer pq)
    m, n, r, K = 12, 10, 3, 2
    cfg, W0 = make([(m, n, r)], K=K, variant=LOCAL)
    o = LordoOracle(cfg, W0)
    per_worker = o.W[0][0].size + o.P[0][0].size + o.u[0][0].size + o.v[0][0].size
    assert per_worker == m * n + m * r + 2 * r * n
    assert o.E[0][0].size == m * n


# ------------------------------------------------------------------ storage rounding modes

def test_bf16_storage_rounds_once_per_step():
    m, n, r = 8, 8, 2
    cfg = OracleConfig(mats=((m, n, r),), K=1, H=1, w_dtype="bf16", e_dtype="bf16", state_dtype="f32")
    W0 = [RNG.standard_normal((m, n)) * 0.02]
    o = LordoOracle(cfg, W0)
    o.inner_step([RNG.standard_normal((1, m, n))], 1e-2, 0.9, 1.0, QHM_NONE)
    for arr in (o.W[0], o.E[0]):
        assert np.array_equal(arr, lo.round_bf16(arr))
    assert np.array_equal(o.u[0], o.u[0].astype(np.float32).astype(np.float64))


# ---------------------------------------------------------------------------------------------
# stored outputs (tests/golden/, written by tests/golden/make_golden.py from the oracle alone)
# ---------------------------------------------------------------------------------------------
def test_golden_files_match_the_oracle():
    """Regression guard, not a pin: the stored values were written by the oracle itself, so this only
    shows that its arithmetic has not changed since (the pins are the other tests of this file)."""
    import importlib.util
    import os
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "make_golden.py"))
    mg = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mg)
    want = np.loadtxt(os.path.join(here, "generator_seed7_purpose2_mat5_index3_replica2_4x8.txt"))
    assert np.array_equal(want, lo.random_matrix(7, 2, 5, 3, 2, 4, 8))
    assert abs(want).max() <= 32 and want.std() > 2.0  # centred Binomial(64, 1/2): sd 4
    for variant, form, name in ((0, 2, "global_fullqhm"), (1, 1, "local_lowqhm")):
        stored = np.loadtxt(os.path.join(here, f"tiny_8x8_{name}_weights.txt"))
        np.testing.assert_allclose(mg.tiny_run(variant, form), stored, rtol=1e-12, atol=1e-15)


# ---------------------------------------------------------------------------------------------
# diagnostics: MSSV of the rotated basis matrix (Sec. "Experimental Framework", Metrics)
# ---------------------------------------------------------------------------------------------
def test_mssv_closed_forms():
    rng = np.random.default_rng(3)
    m, r = 40, 6
    Q, _ = np.linalg.qr(rng.standard_normal((m, 2 * r)))
    A, B = Q[:, :r], Q[:, r:]
    assert abs(lo.mssv(A, A) - 1.0) < 1e-12                      # same subspace: every singular value is 1
    assert abs(lo.mssv(A @ np.linalg.qr(rng.standard_normal((r, r)))[0], A) - 1.0) < 1e-12  # any basis of it
    assert lo.mssv(B, A) < 1e-24                                  # orthogonal subspaces: all zero
    C = np.concatenate([A[:, :3], B[:, :3]], axis=1)              # shares 3 of 6 directions
    assert abs(lo.mssv(C, A) - 0.5) < 1e-12
    # equals ||R||_F^2 / r, the form a kernel would use
    R = C.T @ A
    assert abs(lo.mssv(C, A) - np.sum(R * R) / r) < 1e-12


# ---------------------------------------------------------------------------------------------
# warm-started block power iteration (the alternative ComputeProjection)
# ---------------------------------------------------------------------------------------------
def test_warm_started_power_iteration_pins():
    rng = np.random.default_rng(9)
    m, n, r = 60, 48, 6
    # exact rank r: one iteration from a generic orthonormal start lands on the column space of S
    S = rng.standard_normal((m, r)) @ rng.standard_normal((r, n))
    P0 = np.linalg.qr(rng.standard_normal((m, r)))[0]
    P1 = lo.compute_projection_warm(S, P0, 1)
    assert np.abs(P1.T @ P1 - np.eye(r)).max() < 1e-12
    assert np.linalg.norm(S - P1 @ (P1.T @ S)) / np.linalg.norm(S) < 1e-10
    # a start that already spans the dominant subspace stays there (fixed point up to the basis)
    U, sv, Vt = np.linalg.svd(rng.standard_normal((m, n)), full_matrices=False)
    sv = np.concatenate([np.linspace(10, 5, r), 0.05 * np.ones(len(sv) - r)])
    S = (U * sv) @ Vt
    P2 = lo.compute_projection_warm(S, U[:, :r], 1)
    assert np.linalg.norm(P2 - U[:, :r] @ (U[:, :r].T @ P2), 2) < 1e-10
    # from a generic start the angle to the SVD subspace shrinks like (sigma_{r+1}/sigma_r)^2 per iteration
    angle = lambda P: np.arcsin(min(1.0, np.linalg.norm(P - U[:, :r] @ (U[:, :r].T @ P), 2)))
    a1, a2, a3 = (angle(lo.compute_projection_warm(S, P0, it)) for it in (1, 2, 3))
    assert a2 < a1 * 1e-3 and a3 <= a2 and a1 < 0.2
    # the oracle's refresh uses it when asked to, and draws no sketch
    cfg = lo.OracleConfig(mats=((m, n, r),), K=1, H=1, variant=lo.GLOBAL, warm_start=True, state_dtype="f64", w_dtype="f64", e_dtype="f64")
    orc = lo.LordoOracle(cfg, [np.zeros((m, n))])
    orc.Delta[0] = S
    P_before = orc.P[0].copy()
    orc.refresh_subspace(None)
    assert np.allclose(orc.P[0], lo.compute_projection_warm(S, P_before, 0))


def test_sync_states_is_the_mean_over_workers():
    cfg = lo.OracleConfig(mats=((8, 8, 4),), K=3, H=2, state_dtype="f64", w_dtype="f64", e_dtype="f64")
    orc = lo.LordoOracle(cfg, [np.zeros((8, 8))])
    rng = np.random.default_rng(1)
    orc.u[0] = rng.standard_normal((3, 4, 8)); orc.v[0] = rng.random((3, 4, 8))
    mu, v_before = orc.u[0].mean(axis=0), orc.v[0].copy()
    orc.sync_states(True, False)
    assert np.allclose(orc.u[0], mu[None]) and np.array_equal(orc.v[0], v_before)
    orc.sync_states(False, True)
    assert np.allclose(orc.v[0], v_before.mean(axis=0)[None])


# ---------------------------------------------------------------------------------------------
# Up-link time buffer (App. "Worker Communication"): the pseudo-gradient rebuilt from the low-rank
# accumulators equals the one read off the weights, because every inner step moved the weights by
# exactly eta * Q * alpha (App. "Extended Mathematical Derivations", the telescoped sum).
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("variant", [lo.GLOBAL, lo.LOCAL])
@pytest.mark.parametrize("form", [lo.QHM_NONE, lo.QHM_LOW])
def test_time_buffer_rebuilds_the_dense_pseudo_gradient(variant, form):
    rng = np.random.default_rng(3)
    mats = ((12, 10, 3), (9, 14, 4))
    K, H = 3, 4
    W0 = [rng.standard_normal((m, n)) for m, n, r in mats]
    runs = []
    for tb in (False, True):
        cfg = lo.OracleConfig(mats=mats, K=K, H=H, variant=variant, state_dtype="f64", w_dtype="f64", e_dtype="f64", eps=1e-3,
                              outer=lo.OUTER_NESTEROV, outer_lr=0.7, outer_momentum=0.9, time_buffer=tb)
        orc = lo.LordoOracle(cfg, W0)
        g_rng = np.random.default_rng(4)
        for rnd in range(2):
            for h in range(H):
                G = [g_rng.standard_normal((K, m, n)) for m, n, r in mats]
                if variant == lo.LOCAL and h == 0:
                    orc.refresh_subspace(G, 0.9)
                orc.inner_step(G, 0.01 * (h + 1), 0.9, 0.8, form)  # a different eta every step
            orc.outer_step()
            if variant == lo.GLOBAL:
                orc.refresh_subspace(None, 0.9)
        runs.append(orc)
    dense, tb = runs
    for i in range(len(mats)):
        assert np.allclose(tb.Delta[i], dense.Delta[i], rtol=0, atol=1e-12)
        assert np.allclose(tb.X0[i], dense.X0[i], rtol=0, atol=1e-12)
        assert float(np.abs(tb.T[i]).max()) == 0.0  # cleared by the synchronisation


def test_time_buffer_is_the_sum_of_eta_alpha():
    """One worker, one matrix, no QHM: T after H steps = sum eta_t u^_t / (sqrt(v^_t) + eps), every term
    recomputed here from the low-rank gradients of the run."""
    rng = np.random.default_rng(8)
    m, n, r, H = 7, 6, 2, 3
    cfg = lo.OracleConfig(mats=((m, n, r),), K=1, H=H, variant=lo.GLOBAL, state_dtype="f64", w_dtype="f64", e_dtype="f64",
                          error_feedback=False, eps=1e-2, beta2=0.95, time_buffer=True)
    orc = lo.LordoOracle(cfg, [rng.standard_normal((m, n))])
    P = orc.P[0].copy()
    u = np.zeros((r, n)); v = np.zeros((r, n)); want = np.zeros((r, n))
    for t in range(1, H + 1):
        G = rng.standard_normal((1, m, n))
        eta = 0.1 / t
        orc.inner_step([G], eta, 0.9, 1.0, lo.QHM_NONE)
        g = P.T @ G[0]
        u = 0.9 * u + 0.1 * g
        v = 0.95 * v + 0.05 * g * g
        want += eta * (u / (1 - 0.9 ** t)) / (np.sqrt(v / (1 - 0.95 ** t)) + 1e-2)
    assert np.allclose(orc.T[0][0], want, rtol=1e-12, atol=1e-14)


def test_time_buffer_refuses_what_does_not_factorise():
    cfg = lo.OracleConfig(mats=((6, 6, 2),), K=2, H=2, state_dtype="f64", w_dtype="f64", e_dtype="f64", time_buffer=True)
    orc = lo.LordoOracle(cfg, [np.zeros((6, 6))])
    G = [np.ones((2, 6, 6))]
    with pytest.raises(ValueError):
        orc.inner_step(G, 0.1, 0.9, 0.9, lo.QHM_FULL)
    orc.inner_step(G, 0.1, 0.9, 0.9, lo.QHM_LOW)
    with pytest.raises(ValueError):
        orc.refresh_subspace(None, 0.9)  # the basis may not move inside a round


# ---------------------------------------------------------------------------------------------
# R16: oversampled sketch with Rayleigh-Ritz truncation.
# ---------------------------------------------------------------------------------------------
def _angle(A, B):
    s = np.linalg.svd(np.linalg.qr(A)[0].T @ np.linalg.qr(B)[0], compute_uv=False)
    return float(np.arccos(np.clip(s.min(), -1.0, 1.0)))


def test_rayleigh_ritz_is_the_truncated_svd_of_the_projected_signal():
    """The returned basis spans the top-r left singular vectors of Q Q^T S (numpy's SVD of that matrix)."""
    rng = np.random.default_rng(21)
    m, n, r, p = 40, 30, 5, 4
    S = rng.standard_normal((m, n)) * (0.7 ** np.arange(n))[None, :]
    Om = rng.standard_normal((n, r + p))
    Q = lo.compute_projection(S, Om, 1)
    U = np.linalg.svd(Q @ (Q.T @ S))[0][:, :r]
    P = lo.compute_projection_rr(S, Om, 1, r)
    assert P.shape == (m, r)
    assert np.abs(P.T @ P - np.eye(r)).max() < 1e-12
    assert _angle(P, U) < 1e-6


def test_rayleigh_ritz_recovers_an_exact_rank_r_range_and_beats_the_plain_sketch():
    rng = np.random.default_rng(22)
    m, n, r, p = 36, 28, 4, 4
    L = np.linalg.qr(rng.standard_normal((m, r)))[0]
    S0 = L @ rng.standard_normal((r, n))
    Om = rng.standard_normal((n, r + p))
    assert _angle(lo.compute_projection_rr(S0, Om, 0, r), L) < 1e-7  # exact rank r: the range itself
    # rank r signal + noise: energy captured by r columns, oversampled + truncated vs r-column sketch
    S = S0 + 0.2 * rng.standard_normal((m, n))
    P_rr = lo.compute_projection_rr(S, Om, 0, r)
    P_pl = lo.compute_projection(S, Om[:, :r], 0)
    e_rr, e_pl = np.linalg.norm(P_rr.T @ S), np.linalg.norm(P_pl.T @ S)
    e_best = np.sqrt((np.linalg.svd(S, compute_uv=False)[:r] ** 2).sum())
    assert e_pl < e_rr <= e_best * (1 + 1e-12)


def test_rayleigh_ritz_basis_depends_on_the_subspace_only():
    """Any orthonormal basis of the same (r + p)-dimensional range gives the same P: the eigenvectors'
    signs and order, which a solver is free to choose, do not show in the result."""
    rng = np.random.default_rng(23)
    m, n, r, p = 30, 24, 4, 3
    S = rng.standard_normal((m, n)) * (0.6 ** np.arange(n))[None, :]
    Om = rng.standard_normal((n, r + p))
    P1 = lo.compute_projection_rr(S, Om, 0, r)
    # the same steps with the eigenvectors negated and taken in another order
    Q = lo.compute_projection(S, Om, 0)
    Z = S.T @ Q
    lam, V = np.linalg.eigh(Z.T @ Z)
    Vr = -V[:, np.argsort(lam)[::-1][:r]][:, ::-1]
    P2 = lo.householder_qr_q(Q @ (Vr @ Vr[:r, :].T))
    assert np.abs(P1 - P2).max() < 1e-10


# ---------------------------------------------------------------------------------------------
# Wiring of the refresh and of the driver loop: which basis is "old" and which "new" in the
# rotation, which step count it uses, what the Local signal is, which sketch a refresh draws and
# when a refresh happens. Each test below is built on something fixed outside the oracle: a closed
# form that holds after exactly one moment update, the geometry of a subspace that cannot move, a
# signal whose range is known by construction.
# ---------------------------------------------------------------------------------------------
def _one_step_then_refresh(variant):
    """One worker, one inner step with gradient G1 (so s = 1, E = 0 before it, no clipping), one
    synchronisation, then a refresh that moves the basis. Returns everything a closed form needs."""
    rng = np.random.default_rng(31)
    m, n, r = 24, 18, 4
    b1, b2 = 0.8, 0.95
    cfg, W0 = make([(m, n, r)], K=1, H=1, variant=variant, beta2=b2, eps=1e-3, seed=11)
    o = LordoOracle(cfg, W0)
    G1 = [rng.standard_normal((1, m, n))]
    if variant == LOCAL:
        o.refresh_subspace(G1, b1)  # s = 0: no rotation, only the first basis
    P_old = (o.P[0][0] if variant == LOCAL else o.P[0]).copy()
    o.inner_step(G1, 1e-2, b1, 0.7, QHM_FULL if variant == GLOBAL else QHM_LOW)
    o.outer_step()
    G2 = [rng.standard_normal((1, m, n))]
    o.refresh_subspace(G2 if variant == LOCAL else None, b1)
    P_new = o.P[0][0] if variant == LOCAL else o.P[0]
    return o, P_old, P_new, G1[0][0], b1, b2


@pytest.mark.parametrize("variant", [GLOBAL, LOCAL])
def test_refresh_after_one_step_gives_the_moments_of_that_step_in_the_new_basis(variant):
    """After exactly one moment update u = (1 - b1) g and v = (1 - b2) g o g, so u^ = g and
    v^ - u^ o u^ = 0: the rotation lines of Algorithm 1 then reduce to u' = (1 - b1) g' and
    v' = (1 - b2) g' o g' with g' = P_new^T P_old g, the moments the same step would have left in
    the new basis. The closed form fails if the two bases are swapped in the call (Rot transposed),
    if the rotation is skipped, and if the step count handed to it is not s = 1 (the factor
    (1 - b2^s) / (1 - b1^s)^2 in front of g' o g' is 1 - b2 only for s = 1)."""
    o, P_old, P_new, G1, b1, b2 = _one_step_then_refresh(variant)
    assert subspace_angle(P_old, P_new) > 0.1  # the basis did move
    g = P_old.T @ G1
    g_new = P_new.T @ (P_old @ g)
    assert np.abs(o.u[0][0] - (1 - b1) * g_new).max() < 1e-13
    assert np.abs(o.v[0][0] - (1 - b2) * g_new * g_new).max() < 1e-13
    assert np.abs(o.u[0][0] - (1 - b1) * g).max() > 1e-3  # and differ from the unrotated ones


@pytest.mark.parametrize("variant", [GLOBAL, LOCAL])
def test_refresh_that_cannot_move_the_subspace_keeps_the_first_moment_vector(variant):
    """Stagnation case (Sec. "Enabling Full Subspace Exploration"): the refresh signal has exact rank
    r and lies in span(P), so the new basis spans the same subspace, P_new = P_old Q with Q
    orthogonal, and the first moment, seen in the full space, must not move: P_new u_new = P_old u_old.
    Swapped bases give P_old Q Q u, a skipped rotation P_old Q u."""
    rng = np.random.default_rng(32)
    m, n, r, K = 30, 22, 5, 2
    cfg, W0 = make([(m, n, r)], K=K, H=1, variant=variant, seed=3)
    P0 = np.linalg.qr(rng.standard_normal((m, r)))[0]
    o = LordoOracle(cfg, W0, P0=[P0])
    o.s = 7
    o.u[0] = rng.standard_normal((K, r, n))
    o.v[0] = rng.random((K, r, n)) + 0.5
    u_full = np.stack([P0 @ o.u[0][k] for k in range(K)])
    inside = [P0 @ rng.standard_normal((r, n)) for _ in range(K)]  # rank r, inside span(P)
    if variant == GLOBAL:
        o.Delta[0] = inside[0]
        o.refresh_subspace(None, 0.9)
    else:
        o.refresh_subspace([np.stack(inside)], 0.9)
    for k in range(K):
        P_new = o.P[0][k] if variant == LOCAL else o.P[0]
        assert subspace_angle(P_new, P0) < 1e-7
        assert np.abs(P_new - P0).max() > 1e-2  # another basis of the same subspace
        assert np.abs(P_new @ o.u[0][k] - u_full[k]).max() < 1e-12


def test_local_refresh_signal_is_the_clipped_gradient_plus_the_error_buffer():
    """Algorithm 2, ComputeProjection(G^ + E): with E = L - c G set by hand, L of exact rank r, the
    signal is L whatever G is, and the refresh must return range(L). Dropping E leaves c G (full
    rank), dropping c leaves L + (1 - c) G."""
    rng = np.random.default_rng(33)
    m, n, r, K, rho = 28, 20, 4, 2, 2.0
    cfg, W0 = make([(m, n, r)], K=K, H=1, variant=LOCAL, clip_rho=rho, power_iters=1)
    o = LordoOracle(cfg, W0)
    G = rng.standard_normal((K, m, n))
    L = [np.linalg.qr(rng.standard_normal((m, r)))[0] @ rng.standard_normal((r, n)) for _ in range(K)]
    for k in range(K):
        c = min(1.0, rho / (math.sqrt(float(np.sum(G[k] ** 2))) + 1e-6))
        assert c < 0.2  # the gradient is clipped, so a dropped coefficient shows
        o.E[0][k] = L[k] - c * G[k]
    o.refresh_subspace([G], 0.9)
    for k in range(K):
        P = o.P[0][k]
        assert np.linalg.norm(L[k] - P @ (P.T @ L[k])) / np.linalg.norm(L[k]) < 1e-6
    # without error feedback the signal is the clipped gradient alone: E must then be ignored
    cfg2, _ = make([(m, n, r)], K=K, H=1, variant=LOCAL, clip_rho=rho, error_feedback=False)
    o2 = LordoOracle(cfg2, W0)
    o2.E[0][:] = 5.0 * rng.standard_normal((K, m, n))
    Glow = np.stack([np.linalg.qr(rng.standard_normal((m, r)))[0] @ rng.standard_normal((r, n)) for _ in range(K)])
    o2.refresh_subspace([Glow], 0.9)
    for k in range(K):
        P = o2.P[0][k]
        assert np.linalg.norm(Glow[k] - P @ (P.T @ Glow[k])) / np.linalg.norm(Glow[k]) < 1e-6


@pytest.mark.parametrize("variant", [GLOBAL, LOCAL])
def test_every_refresh_draws_its_own_sketch(variant):
    """The sketch of refresh number j of matrix i (and worker k under the Local rule) is the
    generator's stream (seed, sketch, i, j, k): two refreshes of the same full-rank signal give two
    different bases, each the range finder's answer for its own stream. A refresh counter that
    stands still would repeat the first basis."""
    rng = np.random.default_rng(34)
    mats = [(20, 16, 3), (18, 24, 4)]
    K, seed = 2, 9
    cfg, W0 = make(mats, K=K, H=1, variant=variant, seed=seed)
    o = LordoOracle(cfg, W0)
    S = [rng.standard_normal((K, m, n)) for m, n, _ in mats]
    seen = []
    for j in range(3):
        if variant == GLOBAL:
            for i in range(len(mats)):
                o.Delta[i] = S[i][0]
            o.refresh_subspace(None, 0.9)
        else:
            o.refresh_subspace(S, 0.9)
        for i, (m, n, r) in enumerate(mats):
            for k in range(K if variant == LOCAL else 1):
                Om = lo.random_matrix(seed, lo.PURPOSE_OMEGA, i, j, k, n, r)
                want = np.linalg.qr(S[i][k] @ Om)[0]  # any orthonormal basis of range(S Omega)
                got = o.P[i][k] if variant == LOCAL else o.P[i]
                assert subspace_angle(got, want) < 1e-7, (j, i, k)
        seen.append(np.concatenate([p.ravel() for p in o.P]))
    assert np.abs(seen[0] - seen[1]).max() > 1e-2 and np.abs(seen[1] - seen[2]).max() > 1e-2
    if variant == LOCAL:  # workers draw different sketches
        assert subspace_angle(o.P[0][0], np.linalg.qr(S[0][0] @ lo.random_matrix(seed, lo.PURPOSE_OMEGA, 0, 2, 1, 16, 3))[0]) > 1e-2


def test_driver_loop_refreshes_local_before_the_step_and_global_after_the_sync():
    """R11. Local: the basis is refreshed from the first gradient of a round before that gradient is
    projected, so a gradient of exact rank r is represented without loss and leaves E = 0 (a refresh
    after the step would have projected it onto Q_0 = I[:, :r] and left E != 0). Global: the basis a
    round works with is the range of the previous round's pseudo-gradient, hence after the sync and
    before the next step; with the full-rank QHM term and H = 1 that pseudo-gradient is known in
    closed form from the first basis."""
    rng = np.random.default_rng(35)
    m, n, r, K = 26, 20, 4, 2
    cfg, W0 = make([(m, n, r)], K=K, H=1, variant=LOCAL)
    o = LordoOracle(cfg, W0)
    Glow = np.stack([rng.standard_normal((m, r)) @ rng.standard_normal((r, n)) for _ in range(K)])
    lo.run_rounds(o, lambda rnd, h: [Glow], 1, 1e-2, 0.9, 0.9, QHM_LOW)
    assert np.abs(o.E[0]).max() < 1e-10 * np.abs(Glow).max()
    assert o.refreshes == 1 and o.s == 1
    # Global: two rounds; the second round's low-rank gradient must be taken in the refreshed basis
    cfg, W0 = make([(m, n, r)], K=1, H=1, variant=GLOBAL, seed=4, eps=1e-3)
    o = LordoOracle(cfg, W0)
    P0 = o.P[0].copy()
    G = [rng.standard_normal((1, m, n)) for _ in range(2)]
    lo.run_rounds(o, lambda rnd, h: [G[rnd]], 2, 1e-2, 0.9, 0.5, QHM_FULL)
    assert o.refreshes == 2 and o.s == 2
    # round 1 by hand (s = 1, E = 0, K = 1, averaging outer step): Delta_1 = lr * update
    g = P0.T @ G[0][0]
    D = np.abs(g) + 1e-3                                  # sqrt(v^) + eps with v^ = g o g
    delta1 = 1e-2 * (0.5 * G[0][0] / D.mean(axis=0)[None, :] + 0.5 * P0 @ (g / D))
    P1 = np.linalg.qr(delta1 @ lo.random_matrix(4, lo.PURPOSE_OMEGA, 0, 0, 0, n, r))[0]
    # the error buffer after round 2 is orthogonal to the basis that round 2 projected with
    assert np.abs(P1.T @ o.E[0][0]).max() < 1e-9
    assert np.abs(P0.T @ o.E[0][0]).max() > 1e-3


# ---------------------------------------------------------------------------------------------
# R17: projection from the right (not in the paper). Everything it does is fixed by one identity:
# right-projecting W is left-projecting W^T. The right-side code path of the oracle (g = A Q,
# E = A - g Q^T, p x r moments, row-wise mu, range finder on the transposed signal) is written out on
# its own and compared here with the left-side path, which the tests above pin, on transposed inputs.
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("variant", [GLOBAL, LOCAL])
@pytest.mark.parametrize("form", [QHM_NONE, QHM_LOW, QHM_FULL])
@pytest.mark.parametrize("opts", [dict(), dict(power_iters=1), dict(warm_start=True), dict(error_feedback=False), dict(time_buffer=True)])
def test_right_side_projection_is_left_side_projection_of_the_transpose(variant, form, opts):
    if opts.get("time_buffer") and form == QHM_FULL:
        pytest.skip("the full-rank form does not factorise (R15)")
    rng = np.random.default_rng(41)
    m, n, r, K, H, rounds = 14, 9, 3, 2, 2, 2
    kw = dict(K=K, H=H, variant=variant, clip_rho=1.5, outer=OUTER_NESTEROV, outer_lr=0.7, outer_momentum=0.9, beta2=0.95, eps=1e-4, seed=6,
              state_dtype="f64", w_dtype="f64", e_dtype="f64", **opts)
    W0 = rng.standard_normal((m, n)) * 0.02
    right = LordoOracle(OracleConfig(mats=((m, n, r),), sides=(1,), **kw), [W0])
    left = LordoOracle(OracleConfig(mats=((n, m, r),), sides=(0,), **kw), [W0.T.copy()])
    assert right.P[0].shape == left.P[0].shape  # the basis is q x r on both sides (same generator stream, same shape)
    assert right.u[0].shape == (K, m, r) and left.u[0].shape == (K, r, m)
    grads = [[rng.standard_normal((K, m, n)) * (3.0 if h == 0 else 0.2)] for h in range(H * rounds)]
    lo.run_rounds(right, lambda rnd, h: grads[rnd * H + h], rounds, 0.01, 0.9, 0.7, form)
    lo.run_rounds(left, lambda rnd, h: [np.swapaxes(grads[rnd * H + h][0], 1, 2)], rounds, 0.01, 0.9, 0.7, form)
    T = lambda x: np.swapaxes(x, -1, -2)
    for name in ("W", "E", "u", "v", "X0", "B", "Delta", "T"):
        a, b = getattr(right, name)[0], T(getattr(left, name)[0])
        assert np.abs(a - b).max() <= 1e-12 * max(1.0, np.abs(b).max()), name
    assert np.abs(right.P[0] - left.P[0]).max() < 1e-12
    assert right.refreshes == left.refreshes == rounds
    assert np.abs(right.u[0]).max() > 0 and (not kw.get("error_feedback", True) or np.abs(right.E[0]).max() > 0)


def test_right_side_identity_basis_reduces_to_adam():
    m, n = 11, 6
    cfg, W0 = make([(m, n, n)], K=1, H=1, variant=LOCAL, eps=1e-8, beta2=0.999, sides=(1,))
    o = LordoOracle(cfg, W0)  # Local: Q_0 = I, here the n x n identity applied from the right
    assert o.P[0].shape == (1, n, n)
    grads = [RNG.standard_normal((m, n)) for _ in range(5)]
    for g in grads:
        o.inner_step([g[None]], 3e-3, 0.9, 1.0, QHM_NONE)
    want = _adam_reference(W0[0], grads, 3e-3, 0.9, 0.999, 1e-8)
    assert np.abs(o.W[0][0] - want).max() < 1e-13 and np.abs(o.E[0]).max() == 0.0


def test_right_side_reconstructs_a_gradient_of_low_row_rank():
    m, n, r = 40, 24, 5
    cfg, W0 = make([(m, n, r)], K=1, variant=LOCAL, power_iters=1, sides=(1,))
    o = LordoOracle(cfg, W0)
    G = [(RNG.standard_normal((m, r)) @ RNG.standard_normal((r, n)))[None]]
    o.refresh_subspace(G)
    P = o.P[0][0]
    assert P.shape == (n, r) and np.abs(P.T @ P - np.eye(r)).max() < 1e-10
    assert np.linalg.norm(G[0][0] - (G[0][0] @ P) @ P.T) / np.linalg.norm(G[0][0]) < 1e-6  # the row space is captured
    o.inner_step(G, 1e-3, 0.9, 0.6, QHM_FULL)
    assert np.abs(o.E[0]).max() < 1e-10 * np.abs(G[0]).max()
    # full-rank QHM from the right: one scale per ROW (mean over the rank axis of a p x r array)
    g = G[0][0] @ P
    d = (np.abs(g) + cfg.eps).mean(axis=1)
    upd = 0.4 * G[0][0] / d[:, None] + 0.6 * ((g / (np.abs(g) + cfg.eps)) @ P.T)
    assert np.abs(o.W[0][0] - (W0[0] - 1e-3 * upd)).max() < 1e-12
