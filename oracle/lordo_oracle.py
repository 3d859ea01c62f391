"""CPU oracle for the LoRDO optimizer hot path. TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 restatement of what the path computes, written from the paper's definitions
(Algorithm 1 = Global variant, Algorithm 2 = Local variant, Sec. "Low-Rank Adaptive Optimization",
Sec. "Enabling Full Subspace Exploration", App. "Extended Mathematical Derivations"). It shares no
code with the CUDA path and must never be imported by the product: only the tests, the smoke
check and the benchmark's cpu baseline leg may call it.

Arithmetic is numpy float64; `numpy.matmul` and nothing else from a library serves as a step.
Stored state is rounded to the storage type of the configuration after every update (fp32 for the
moments, projection, anchor, outer momentum; fp32 or bf16 for weights and the error buffer), or
kept in fp64 when ``state_dtype="f64"`` (used by the mathematical pins).

Readings of points the paper leaves open (each is restated where it is used):
  R1  ComputeProjection is a randomized range finder: sketch width exactly r, `power_iters`
      subspace iterations, thin Householder QR with diag(R) >= 0 after every product. The paper's
      definition (top-r left singular vectors, Sec. 2) is the target it approximates.
  R2  The projection is always applied from the left (Q is p x r, moments are r x q; Sec. 2).
  R3  Bias correction is Adam's, with the global count s of moment updates, never reset
      (the algorithms' captions say it is omitted from the notation only).
  R4  The power of beta_2 in the second-moment rotation is that same s; no rotation at s = 0.
  R5  "(Q'^T Q)^2" in the second-moment rotation is the element-wise square (LDAdam's rule).
  R6  mu(z) = (1/r) sum_i z_i runs over the rank axis: one scale per column.
  R7  Full-rank QHM uses the clipped gradient without the error buffer.
  R8  Clipping: one L2 norm per worker over all matrices, coefficient min(1, rho/(norm+1e-6)).
  R9  Pseudo-gradient sign follows the appendix: Delta = old - new, theta <- theta - eta_s Delta.
  R10 Nesterov outer step: B <- mu B + Delta ; theta <- theta - eta_s (Delta + mu B).
  R11 A round is H inner steps then a sync. Global refreshes right after the sync from Delta;
      Local refreshes at the first step of every round from that step's c*G + E.
  R12 Q_0: Global = orthonormalised random matrix; Local = first r columns of the identity.
  R13 The error buffer is left untouched by a refresh; there is no weight decay.
  R14 Random matrices come from a counter-based integer generator (below): entries are
      popcount(64-bit word) - 32, i.e. centred Binomial(64, 1/2) integers, variance 16.
  R16 Oversampled sketch (`oversample` = p > 0): the range finder runs with r + p columns and the
      basis is truncated to the top-r left singular subspace of its projection of the signal
      (Rayleigh-Ritz), see compute_projection_rr. Not in the paper: the randomized-SVD refinement of
      R1, closer to the paper's SVD definition of the projection at the same rank.
  R17 Right-side projection (`sides[i] = 1`; not in the paper, which always projects from the left: the
      side selection of GaLore-type methods for matrices with more rows than columns): the basis Q is
      q x r, the low-rank gradient is g = (G^ + E) Q (p x r), the moments are p x r, the update is
      U~ Q^T, the full-rank QHM scale mu(.) runs over the rank axis and gives one value per row, and
      ComputeProjection returns the top-r right singular subspace (the range finder applied to the
      transposed signal, sketch p x r). Everything equals the left-side method applied to W^T.
  R15 Up-link time buffer (App. "Worker Communication", the server-side repacked updates): with
      `time_buffer` every worker accumulates T <- T + eta * alpha, alpha being the low-rank update of
      the step (no QHM or low-rank QHM only), and the pseudo-gradient of the synchronisation is
      rebuilt as Delta = (1/M) sum_m Q^m T^m instead of being read off the weights; T is cleared
      after every synchronisation. The basis must stay fixed between two synchronisations.

Parity status: every function here is pinned by tests/test_oracle_pins.py against closed forms,
invariants, library routines (torch.optim.Adam / SGD, numpy.linalg.svd / qr) or brute force; the
wiring of refresh_subspace and run_rounds (which basis is old and which new in the rotation, the
step count it uses, the Local signal, the sketch index, when a refresh happens) by closed forms
that hold after one moment update, by a subspace that cannot move and by signals of known range.
Agreement with the authors' own (unpublished) code on R1-R16 is "parity unpinned".
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence, Tuple

import numpy as np

GLOBAL, LOCAL = 0, 1
QHM_NONE, QHM_LOW, QHM_FULL = 0, 1, 2
OUTER_AVG, OUTER_NESTEROV = 0, 1

PURPOSE_P0, PURPOSE_OMEGA = 1, 2

_MASK = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15


# ----------------------------------------------------------------------------------------------
# R14: counter-based integer generator (integers only, so host and device agree bit for bit)
# ----------------------------------------------------------------------------------------------

def mix64_int(x: int) -> int:
    """The splitmix64 output permutation on one python integer."""
    x &= _MASK
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _MASK
    return x ^ (x >> 31)


def stream_key(seed: int, purpose: int, mat: int, index: int, replica: int) -> int:
    """Key of one random matrix: chained mixes of (seed, purpose, matrix id, draw index, replica)."""
    k = mix64_int(seed + _GOLDEN)
    for field in (purpose, mat, index, replica):
        k = mix64_int((k + _GOLDEN * (field + 1)) & _MASK)
    return k


def _mix64_vec(x: np.ndarray) -> np.ndarray:
    x = x.astype(np.uint64, copy=True)
    x ^= x >> np.uint64(30)
    x *= np.uint64(0xBF58476D1CE4E5B9)
    x ^= x >> np.uint64(27)
    x *= np.uint64(0x94D049BB133111EB)
    x ^= x >> np.uint64(31)
    return x


def random_words(key: int, count: int) -> np.ndarray:
    """word[c] = mix64(key + GOLDEN * (c + 1)) for c = 0..count-1 (uint64)."""
    with np.errstate(over="ignore"):
        c = np.arange(1, count + 1, dtype=np.uint64) * np.uint64(_GOLDEN) + np.uint64(key)
        return _mix64_vec(c)


def popcount64(w: np.ndarray) -> np.ndarray:
    w = w.astype(np.uint64, copy=True)
    m1, m2, m4 = np.uint64(0x5555555555555555), np.uint64(0x3333333333333333), np.uint64(0x0F0F0F0F0F0F0F0F)
    w = w - ((w >> np.uint64(1)) & m1)
    w = (w & m2) + ((w >> np.uint64(2)) & m2)
    w = (w + (w >> np.uint64(4))) & m4
    with np.errstate(over="ignore"):
        w = (w * np.uint64(0x0101010101010101)) >> np.uint64(56)
    return w.astype(np.int64)


def random_matrix(seed: int, purpose: int, mat: int, index: int, replica: int, rows: int, cols: int) -> np.ndarray:
    """rows x cols matrix of centred Binomial(64,1/2) integers (as float64), row-major counter."""
    words = random_words(stream_key(seed, purpose, mat, index, replica), rows * cols)
    return (popcount64(words) - 32).astype(np.float64).reshape(rows, cols)


# ----------------------------------------------------------------------------------------------
# storage rounding
# ----------------------------------------------------------------------------------------------

def round_bf16(x: np.ndarray) -> np.ndarray:
    """fp64/fp32 -> nearest fp32 -> nearest-even bf16, returned as float64."""
    f = np.asarray(x, dtype=np.float32)
    bits = f.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    rounded = ((bits + np.uint64(0x7FFF) + lsb) >> np.uint64(16)) << np.uint64(16)
    out = (rounded & np.uint64(0xFFFFFFFF)).astype(np.uint32).view(np.float32)
    out = np.where(np.isfinite(f), out, f)
    return out.astype(np.float64)


def store(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "f64":
        return np.asarray(x, dtype=np.float64)
    if dtype == "f32":
        return np.asarray(x, dtype=np.float32).astype(np.float64)
    if dtype == "bf16":
        return round_bf16(x)
    raise ValueError(dtype)


# ----------------------------------------------------------------------------------------------
# linear algebra steps
# ----------------------------------------------------------------------------------------------

def householder_qr_q(Y: np.ndarray) -> np.ndarray:
    """Thin Q factor (rows x r, rows >= r) of Y by Householder reflections, signs fixed so that
    diag(R) >= 0. R1: the orthonormal basis of an r-column matrix (Sec. 2: Q = U[:, :r] is
    orthonormal)."""
    A = np.array(Y, dtype=np.float64, copy=True)
    rows, r = A.shape
    assert rows >= r
    V = np.zeros((rows, r))
    diag_sign = np.ones(r)
    for j in range(r):
        x = A[j:, j]
        normx = np.sqrt(np.dot(x, x))
        v = x.copy()
        if normx == 0.0:
            v[0] = 1.0  # degenerate column: any unit vector; reflector e_j keeps the recursion going
            alpha = 0.0
        else:
            alpha = -normx if x[0] >= 0 else normx  # R_jj = alpha
            v[0] -= alpha
        vn = np.sqrt(np.dot(v, v))
        if vn > 0:
            v /= vn
        V[j:, j] = v
        A[j:, j:] -= 2.0 * np.outer(v, v @ A[j:, j:])
        diag_sign[j] = -1.0 if alpha < 0 else 1.0
    Q = np.zeros((rows, r))
    Q[:r, :r] = np.eye(r)
    for j in range(r - 1, -1, -1):
        v = V[j:, j]
        Q[j:, :] -= 2.0 * np.outer(v, v @ Q[j:, :])
    return Q * diag_sign[None, :]


def compute_projection(S: np.ndarray, Omega: np.ndarray, power_iters: int) -> np.ndarray:
    """R1: randomized range finder for the top-r left subspace of S (m x n) with sketch Omega
    (n x r): P' = qr(S Omega); then `power_iters` times Z = qr(S^T P'), P' = qr(S Z)."""
    S = np.asarray(S, dtype=np.float64)
    Pn = householder_qr_q(S @ Omega)
    for _ in range(power_iters):
        Z = householder_qr_q(S.T @ Pn)
        Pn = householder_qr_q(S @ Z)
    return Pn


def compute_projection_rr(S: np.ndarray, Omega: np.ndarray, power_iters: int, r: int) -> np.ndarray:
    """R16: range finder with an oversampled sketch (Omega is n x (r + p)) and Rayleigh-Ritz truncation
    back to rank r. Q = the range finder's (r + p)-column basis; the top-r left singular subspace of
    Q Q^T S is Q V_r, V_r the eigenvectors of the r largest eigenvalues of (Q^T S)(Q^T S)^T
    (`numpy.linalg.eigh` serves as that step). A basis of a subspace is not unique, and the moments
    live in the basis's coordinates, so the basis returned is fixed by the subspace alone:
    P' = qr(Q M[:, :r]) with the projector M = V_r V_r^T."""
    S = np.asarray(S, dtype=np.float64)
    Q = compute_projection(S, Omega, power_iters)          # m x (r + p), orthonormal
    Z = S.T @ Q                                            # n x (r + p)
    lam, V = np.linalg.eigh(Z.T @ Z)                       # ascending eigenvalues
    Vr = V[:, np.argsort(lam)[::-1][:r]]                   # (r + p) x r
    M_r = Vr @ Vr[:r, :].T                                 # first r columns of the projector V_r V_r^T
    return householder_qr_q(Q @ M_r)


def compute_projection_warm(S: np.ndarray, P_old: np.ndarray, iters: int) -> np.ndarray:
    """Block power iteration started from the previous basis (the cheaper ComputeProjection the paper
    names, Sec. 2 "PowerSGD / block power iteration" and App. "Limitations"): `iters` >= 1 times
    Z = qr(S^T P'), P' = qr(S Z), beginning with P' = P_old. No random sketch is drawn."""
    S = np.asarray(S, dtype=np.float64)
    Pn = np.asarray(P_old, dtype=np.float64)
    for _ in range(max(int(iters), 1)):
        Z = householder_qr_q(S.T @ Pn)
        Pn = householder_qr_q(S @ Z)
    return Pn


def rotate_moments(u: np.ndarray, v: np.ndarray, P_new: np.ndarray, P_old: np.ndarray, beta1: float,
                   beta2: float, s: int) -> Tuple[np.ndarray, np.ndarray]:
    """Algorithm 1, moment-rotation lines (same in Algorithm 2). Rot = P_new^T P_old (r x r);
    u <- Rot u ; v <- (1 - beta2^s) | (Rot o Rot)(v_hat - u_hat o u_hat) + (Rot u_hat) o (Rot u_hat) |
    with the bias-corrected u_hat, v_hat of the moments before rotation (R3, R4, R5)."""
    Rot = P_new.T @ P_old
    u_hat = u / (1.0 - beta1 ** s)
    v_hat = v / (1.0 - beta2 ** s)
    ru = Rot @ u_hat
    v_new = (1.0 - beta2 ** s) * np.abs((Rot * Rot) @ (v_hat - u_hat * u_hat) + ru * ru)
    u_new = Rot @ u
    return u_new, v_new


def mssv(P_new: np.ndarray, P_old: np.ndarray) -> float:
    """Sec. "Experimental Framework", Metrics: mean squared singular value of the rotated basis
    matrix R = Q_t^T Q_{t-1}, MSSV = (1/r) sum_i sigma_i^2, written out from the singular values."""
    sigma = np.linalg.svd(np.asarray(P_new, dtype=np.float64).T @ np.asarray(P_old, dtype=np.float64), compute_uv=False)
    return float(np.sum(sigma ** 2) / len(sigma))


def clip_coefficients(G: Sequence[np.ndarray], rho: float, scope: int = 0) -> np.ndarray:
    """R8 / Algorithm 1 line "clip": coefficient per worker (scope 0: one norm over all matrices of
    the worker; scope 1: one per matrix). G[i] has shape [K, m_i, n_i]. Returns [n_mats, K]."""
    n_mats, K = len(G), G[0].shape[0]
    if rho is None or rho <= 0:
        return np.ones((n_mats, K))
    sq = np.array([[np.sum(np.asarray(G[i][k], dtype=np.float64) ** 2) for k in range(K)] for i in range(n_mats)])
    if scope == 0:
        norm = np.sqrt(sq.sum(axis=0, keepdims=True)).repeat(n_mats, axis=0)
    else:
        norm = np.sqrt(sq)
    return np.minimum(1.0, rho / (norm + 1e-6))


# ----------------------------------------------------------------------------------------------
# the four verbs
# ----------------------------------------------------------------------------------------------

@dataclasses.dataclass
class OracleConfig:
    mats: Tuple[Tuple[int, int, int], ...]
    K: int
    H: int
    variant: int = GLOBAL
    error_feedback: bool = True
    beta2: float = 0.999
    eps: float = 1e-8
    clip_rho: float = 0.0
    clip_scope: int = 0
    sync_u: bool = True
    sync_v: bool = True
    outer: int = OUTER_AVG
    outer_lr: float = 1.0
    outer_momentum: float = 0.0
    power_iters: int = 0
    seed: int = 0
    w_dtype: str = "f32"
    e_dtype: str = "f32"
    state_dtype: str = "f32"  # u, v, P, X0, B, Delta
    warm_start: bool = False   # refresh by block power iteration from the current P (no sketch)
    time_buffer: bool = False  # R15: pseudo-gradient rebuilt from the accumulated low-rank updates
    oversample: int = 0        # R16: extra sketch columns p, Rayleigh-Ritz truncation back to rank r
    sides: Optional[Tuple[int, ...]] = None  # R17: per matrix, 0 = project from the left (the paper), 1 = from the right


class LordoOracle:
    """State of all matrices and replicas plus init / inner_step / outer_step / refresh_subspace."""

    def __init__(self, cfg: OracleConfig, W0: Sequence[np.ndarray], P0: Optional[Sequence[np.ndarray]] = None):
        self.cfg = cfg
        c = cfg
        self.s = 0  # moment updates done so far (R3)
        self.refreshes = 0
        self.W, self.E, self.P, self.u, self.v, self.X0, self.B, self.Delta = [], [], [], [], [], [], [], []
        self.T = []  # R15: accumulated eta * alpha per worker, r x n
        self.steps_in_round = 0
        self.last_clip = None
        self.last_mssv = None  # [n_mats][1 or K] MSSV of the last refresh that rotated (diagnostic)
        for i, (m, n, r) in enumerate(c.mats):
            w0 = store(W0[i], c.w_dtype)
            self.W.append(np.repeat(w0[None], c.K, axis=0))  # all workers start equal (Alg. 1 Require)
            self.E.append(np.zeros((c.K, m, n)))
            right = self.side(i) == 1
            lowrank = (c.K, m, r) if right else (c.K, r, n)  # R17: moments are p x r when projecting from the right
            self.u.append(np.zeros(lowrank))
            self.v.append(np.zeros(lowrank))
            self.T.append(np.zeros(lowrank))
            self.X0.append(store(w0, c.state_dtype))
            self.B.append(np.zeros((m, n)))
            self.Delta.append(np.zeros((m, n)))
            pm = n if right else m  # rows of the basis
            if P0 is not None:
                p = np.asarray(P0[i], dtype=np.float64)
            elif c.variant == GLOBAL:
                # R12: random initial projection, orthonormalised
                p = householder_qr_q(random_matrix(c.seed, PURPOSE_P0, i, 0, 0, pm, r))
            else:
                p = np.eye(pm, r)  # R12: Q_0 = identity (Algorithm 2 Require)
            if c.variant == LOCAL and p.ndim == 2:
                p = np.repeat(p[None], c.K, axis=0)
            self.P.append(store(p, c.state_dtype))

    def _P(self, i: int, k: int) -> np.ndarray:
        return self.P[i][k] if self.cfg.variant == LOCAL else self.P[i]

    def side(self, i: int) -> int:
        return 0 if self.cfg.sides is None else int(self.cfg.sides[i])

    # -- Algorithm 1 / 2, the per-step block ------------------------------------------------------
    def inner_step(self, G: Sequence[np.ndarray], lr: float, beta1: float, omega: float, form: int) -> None:
        c = self.cfg
        self.s += 1
        s = self.s
        coef = clip_coefficients(G, c.clip_rho, c.clip_scope)
        self.last_clip = coef
        bc1 = 1.0 - beta1 ** s
        bc2 = 1.0 - c.beta2 ** s
        if c.time_buffer and form == QHM_FULL:
            raise ValueError("the full-rank QHM update has no low-rank factorisation (R15)")
        self.steps_in_round += 1
        for i, (m, n, r) in enumerate(c.mats):
            for k in range(c.K):
                P = self._P(i, k)
                Ghat = coef[i, k] * np.asarray(G[i][k], dtype=np.float64)  # clipped gradient
                A = Ghat + self.E[i][k] if c.error_feedback else Ghat
                if self.side(i) == 1:
                    self._inner_right(i, k, P, Ghat, A, lr, beta1, omega, form, bc1, bc2)
                    continue
                g = P.T @ A  # low-rank gradient with error feedback
                if c.error_feedback:
                    self.E[i][k] = store(A - P @ g, c.e_dtype)
                u = beta1 * self.u[i][k] + (1.0 - beta1) * g
                v = c.beta2 * self.v[i][k] + (1.0 - c.beta2) * g * g
                self.u[i][k] = store(u, c.state_dtype)
                self.v[i][k] = store(v, c.state_dtype)
                u_hat = self.u[i][k] / bc1
                v_hat = self.v[i][k] / bc2
                D = np.sqrt(v_hat) + c.eps
                if form == QHM_NONE:
                    alpha = u_hat / D
                    upd = P @ alpha
                elif form == QHM_LOW:
                    alpha = (omega * u_hat + (1.0 - omega) * g) / D
                    upd = P @ alpha
                elif form == QHM_FULL:
                    d = D.mean(axis=0)  # R6: mean over the rank axis, one value per column
                    upd = (1.0 - omega) * Ghat / d[None, :] + omega * (P @ (u_hat / D))  # R7
                else:
                    raise ValueError(form)
                self.W[i][k] = store(self.W[i][k] - lr * upd, c.w_dtype)
                if c.time_buffer:
                    self.T[i][k] = store(self.T[i][k] + lr * alpha, c.state_dtype)

    def _inner_right(self, i, k, P, Ghat, A, lr, beta1, omega, form, bc1, bc2) -> None:
        """R17: the per-step lines of Algorithm 1 with the basis applied from the right (P is q x r)."""
        c = self.cfg
        g = A @ P  # p x r
        if c.error_feedback:
            self.E[i][k] = store(A - g @ P.T, c.e_dtype)
        u = beta1 * self.u[i][k] + (1.0 - beta1) * g
        v = c.beta2 * self.v[i][k] + (1.0 - c.beta2) * g * g
        self.u[i][k] = store(u, c.state_dtype)
        self.v[i][k] = store(v, c.state_dtype)
        u_hat = self.u[i][k] / bc1
        v_hat = self.v[i][k] / bc2
        D = np.sqrt(v_hat) + c.eps
        if form == QHM_NONE:
            alpha = u_hat / D
            upd = alpha @ P.T
        elif form == QHM_LOW:
            alpha = (omega * u_hat + (1.0 - omega) * g) / D
            upd = alpha @ P.T
        elif form == QHM_FULL:
            d = D.mean(axis=1)  # R6 with R17: mean over the rank axis, one value per row
            upd = (1.0 - omega) * Ghat / d[:, None] + omega * ((u_hat / D) @ P.T)
        else:
            raise ValueError(form)
        self.W[i][k] = store(self.W[i][k] - lr * upd, c.w_dtype)
        if c.time_buffer:
            self.T[i][k] = store(self.T[i][k] + lr * alpha, c.state_dtype)

    # -- Algorithm 1, the two state-synchronisation lines on their own (K_u, K_v != K_x) ------------
    def sync_states(self, sync_u: bool, sync_v: bool) -> None:
        c = self.cfg
        for i in range(len(c.mats)):
            if sync_u:
                self.u[i][:] = store(self.u[i].mean(axis=0), c.state_dtype)[None]
            if sync_v:
                self.v[i][:] = store(self.v[i].mean(axis=0), c.state_dtype)[None]

    # -- Algorithm 1, the synchronisation block ---------------------------------------------------
    def outer_step(self) -> None:
        c = self.cfg
        for i in range(len(c.mats)):
            if c.sync_u:
                self.u[i][:] = store(self.u[i].mean(axis=0), c.state_dtype)[None]
            if c.sync_v:
                self.v[i][:] = store(self.v[i].mean(axis=0), c.state_dtype)[None]
            if c.time_buffer:  # R15: (1/M) sum_m Q^m T^m
                if self.side(i) == 1:
                    delta = np.mean([self.T[i][k] @ self._P(i, k).T for k in range(c.K)], axis=0)
                else:
                    delta = np.mean([self._P(i, k) @ self.T[i][k] for k in range(c.K)], axis=0)
                self.T[i][:] = 0.0
            else:
                delta = self.X0[i] - self.W[i].mean(axis=0)  # R9
            if c.outer == OUTER_AVG:
                x_new = self.X0[i] - delta
            else:  # R10
                self.B[i] = store(c.outer_momentum * self.B[i] + delta, c.state_dtype)
                x_new = self.X0[i] - c.outer_lr * (delta + c.outer_momentum * self.B[i])
            self.Delta[i] = store(delta, c.state_dtype)
            self.X0[i] = store(x_new, c.state_dtype)
            self.W[i][:] = store(self.X0[i], c.w_dtype)[None]
        self.steps_in_round = 0

    # -- ComputeProjection + moment rotation ------------------------------------------------------
    def refresh_subspace(self, G: Optional[Sequence[np.ndarray]] = None, beta1: float = 0.9) -> None:
        c = self.cfg
        if c.time_buffer and self.steps_in_round > 0:
            raise ValueError("the basis must stay fixed between two synchronisations (R15)")
        coef = None
        if c.variant == LOCAL:
            assert G is not None
            coef = clip_coefficients(G, c.clip_rho, c.clip_scope)
        diag = [[] for _ in c.mats]
        for i, (m, n, r) in enumerate(c.mats):
            right = self.side(i) == 1
            for k in range(c.K if c.variant == LOCAL else 1):
                if c.variant == GLOBAL:
                    S = self.Delta[i]                                          # Algorithm 1: ComputeProjection(Delta)
                    P_old = self.P[i]
                else:
                    S = coef[i, k] * np.asarray(G[i][k], dtype=np.float64)     # Algorithm 2: ComputeProjection(G^ + E)
                    if c.error_feedback:
                        S = S + self.E[i][k]
                    P_old = self.P[i][k]
                if right:
                    S = S.T  # R17: the right singular subspace of S is the left one of S^T
                cols = S.shape[1]
                if c.warm_start:
                    P_new = store(compute_projection_warm(S, P_old, c.power_iters), c.state_dtype)
                else:
                    Om = random_matrix(c.seed, PURPOSE_OMEGA, i, self.refreshes, k, cols, r + c.oversample)
                    if c.oversample:
                        P_new = store(compute_projection_rr(S, Om, c.power_iters, r), c.state_dtype)
                    else:
                        P_new = store(compute_projection(S, Om, c.power_iters), c.state_dtype)
                diag[i].append(mssv(P_new, P_old))
                if self.s > 0:
                    for kk in (range(c.K) if c.variant == GLOBAL else (k,)):
                        if right:  # the moments are p x r: their transposes are rotated like left-side moments
                            un, vn = rotate_moments(self.u[i][kk].T, self.v[i][kk].T, P_new, P_old, beta1, c.beta2, self.s)
                            un, vn = un.T, vn.T
                        else:
                            un, vn = rotate_moments(self.u[i][kk], self.v[i][kk], P_new, P_old, beta1, c.beta2, self.s)
                        self.u[i][kk] = store(un, c.state_dtype)
                        self.v[i][kk] = store(vn, c.state_dtype)
                if c.variant == GLOBAL:
                    self.P[i] = P_new
                else:
                    self.P[i][k] = P_new
        self.last_mssv = diag
        self.refreshes += 1


def run_rounds(orc: LordoOracle, grad_fn, rounds: int, lr: float, beta1: float, omega: float, form: int,
               refresh: bool = True) -> None:
    """R11: the driver loop. grad_fn(round, step) -> list over matrices of [K, m, n] arrays."""
    c = orc.cfg
    for rnd in range(rounds):
        for h in range(c.H):
            G = grad_fn(rnd, h)
            if refresh and c.variant == LOCAL and h == 0:
                orc.refresh_subspace(G, beta1)
            orc.inner_step(G, lr, beta1, omega, form)
        orc.outer_step()
        if refresh and c.variant == GLOBAL:
            orc.refresh_subspace(None, beta1)
