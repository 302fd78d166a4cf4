"""CPU oracle for ARMOR's per-layer block coordinate descent.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 restatement of what the ARMOR paper (arXiv 2510.05528)
computes for one linear layer, written step by step from the paper's equations
and algorithms.  It exists to check the CUDA library; it shares no code with
it, is never imported by it, and is not a fallback for it.  Only the test
suite, the smoke check and the benchmark's CPU-baseline leg may call it.

Notation (Section 3.1): W is the (optionally normalised) weight
[d_out, d_in]; A, B are block-diagonal wrappers stored as [nb, d_block,
d_block]; S = W' (.) M is the N:M-sparse core; M is a boolean array; the
reconstruction is  W_hat = A S B  (the factorisation of Section 3.1).  X is [n_tokens, d_in] (the paper's
X^T, Section 2), H = X^T X, and H_w is the weighting of the proxy loss:
  h_mode = DIAG : H_w = diag(H)    -- the paper's loss, Eq. proxy_loss
  h_mode = FULL : H_w = H          -- the full-Gram generalisation
                                      L = tr(E H_w E^T),  E = W - A S B.
Everything below is written for a general symmetric PSD H_w; with a diagonal
H_w every formula reduces to the paper's.

Equations are cited by the paper's own labels (proxy_loss, init, proxyBlock,
mask_loss_opt, mask_loss_opt_sol, lrA, lrB, lrWprime) because its printed
cross-references use two numberings.  Readings of points the paper leaves
open are marked "Reading:".
Parity status: every function here is pinned by tests/test_oracle_*.py to
closed forms, brute force, textbook least squares or the paper's theorems.
The final iterates on the benchmark configurations have no printed
counterpart in the paper: *parity unpinned* for those values as such; they
are constrained only by the invariants (monotone loss, L_t <= L_0, ...).
"""
from __future__ import annotations

import itertools
from dataclasses import dataclass, field

import numpy as np

FULL, DIAG = 0, 1
L1_RANDOM, L1_GREEDY, UNIFORM_RANDOM, L2_RANDOM = 0, 1, 2, 3
S_EXACT, S_BETA = 0, 1
AB_EXACT, AB_GD, AB_ADAM = 0, 1, 2
PH_A, PH_B, PH_S, PH_MASK = 1, 2, 4, 8
PH_ALL = 15


@dataclass
class OracleConfig:
    d_block: int
    n_keep: int = 2
    m_group: int = 4
    h_mode: int = FULL
    select_mode: int = L1_RANDOM
    s_step: int = S_EXACT
    ab_step: int = AB_EXACT
    adam_lr: float = 1e-4          # Appendix F
    adam_beta1: float = 0.9        # Reading: the defaults of Kingma & Ba, which the paper cites without values
    adam_beta2: float = 0.999
    adam_eps: float = 1e-8
    ridge: float = 1e-6
    seed: int = 0
    phases: int = PH_ALL
    mask_sweeps: int = 1         # sparse-core updates (Algorithm 3) per continuous update; the paper runs 1
    mask_groups: int = 1         # groups drawn per block in one sparse-core update; the paper draws 1


@dataclass
class IterInfo:
    """What one iteration did (diagnostics; the margins feed the parity tests)."""
    loss: dict = field(default_factory=dict)       # loss after each sub-step
    tau_A: float = 0.0
    tau_B: float = 0.0
    tau_S: float = 0.0
    chol_failed: int = 0
    groups_changed: int = 0
    mask_accepted: int = 1
    delta_L_mask: float = 0.0
    selected: np.ndarray | None = None             # [nbo, nbi] global group index or -1
    select_margin: np.ndarray | None = None        # [nbo, nbi] relative margin of the selection
    mask_margin: np.ndarray | None = None          # [nbo, nbi] relative margin of the mask sweep
    new_mask: np.ndarray | None = None             # [nbo, nbi] chosen mask byte
    sweeps: list = field(default_factory=list)     # one IterInfo per sparse-core update of the iteration
    selected_all: np.ndarray | None = None         # [nbo, nbi, mask_groups] every group drawn, -1 where none


# --------------------------------------------------------------------------
# block-diagonal helpers: the definition of a product with diag(A_1..A_nb)
# --------------------------------------------------------------------------
def bd_left(Ablk: np.ndarray, Y: np.ndarray) -> np.ndarray:
    """diag(A_1..A_nb) @ Y ; row-block i of the result is A_i @ Y_i (Section 3.1)."""
    nb, db, _ = Ablk.shape
    out = np.empty_like(Y, dtype=np.float64)
    for i in range(nb):
        out[i * db:(i + 1) * db] = Ablk[i] @ Y[i * db:(i + 1) * db]
    return out


def bd_right(Y: np.ndarray, Bblk: np.ndarray) -> np.ndarray:
    """Y @ diag(B_1..B_nb) ; column-block j of the result is Y_j @ B_j."""
    nb, db, _ = Bblk.shape
    out = np.empty_like(Y, dtype=np.float64)
    for j in range(nb):
        out[:, j * db:(j + 1) * db] = Y[:, j * db:(j + 1) * db] @ Bblk[j]
    return out


def bd_T(Ablk: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(np.transpose(Ablk, (0, 2, 1)))


def bd_dense(Ablk: np.ndarray) -> np.ndarray:
    """The block-diagonal matrix written out densely (small cases only)."""
    nb, db, _ = Ablk.shape
    out = np.zeros((nb * db, nb * db))
    for i in range(nb):
        out[i * db:(i + 1) * db, i * db:(i + 1) * db] = Ablk[i]
    return out


# --------------------------------------------------------------------------
# O0  calibration statistics
# --------------------------------------------------------------------------
def gram(X: np.ndarray, H: np.ndarray | None = None) -> np.ndarray:
    """H (+)= X^T X.  Its diagonal is ||X_j||^2, the weight of Eq. proxy_loss."""
    X64 = np.asarray(X, dtype=np.float64)
    G = X64.T @ X64
    return G if H is None else H + G


def weighting(H: np.ndarray, h_mode: int) -> np.ndarray:
    H = np.asarray(H, dtype=np.float64)
    if h_mode == DIAG:
        return np.diag(np.diag(H))
    return H


# --------------------------------------------------------------------------
# O1  NoWag normalisation (Section 3.2, the display after Eq. proxy_loss)
# --------------------------------------------------------------------------
def normalize(W: np.ndarray):
    """W_bar_ij = W_ij / r1_j / r2_i with r1 the column norms of W and r2 the
    row norms of W / r1.  Reading: a zero norm is replaced by 1."""
    W = np.asarray(W, dtype=np.float64)
    r1 = np.sqrt((W * W).sum(axis=0))
    r1 = np.where(r1 == 0.0, 1.0, r1)
    Wc = W / r1[None, :]
    r2 = np.sqrt((Wc * Wc).sum(axis=1))
    r2 = np.where(r2 == 0.0, 1.0, r2)
    return Wc / r2[:, None], r1, r2


# --------------------------------------------------------------------------
# O2  initialisation (Eq. init, Section 3.3)
# --------------------------------------------------------------------------
def init(W: np.ndarray, H: np.ndarray, cfg: OracleConfig):
    """A = B = I, W' = W, M = top-n of every group of m by W_ij^2 * H_jj.
    Reading: ties keep the lower column index.  The score always uses diag(H)."""
    W = np.asarray(W, dtype=np.float64)
    d_out, d_in = W.shape
    db, n, m = cfg.d_block, cfg.n_keep, cfg.m_group
    score = W * W * np.diag(H)[None, :]
    M = np.zeros((d_out, d_in), dtype=bool)
    sg = score.reshape(d_out, d_in // m, m)
    # stable sort of (-score): equal scores keep ascending column order
    order = np.argsort(-sg, axis=2, kind="stable")[:, :, :n]
    Mg = M.reshape(d_out, d_in // m, m)
    np.put_along_axis(Mg, order, True, axis=2)
    A = np.tile(np.eye(db), (d_out // db, 1, 1))
    B = np.tile(np.eye(db), (d_in // db, 1, 1))
    S = W * M
    return A, B, S, M


def pack_mask(M: np.ndarray, m_group: int = 4) -> np.ndarray:
    """One byte per group; bit p set <=> column m*c + p is kept."""
    d_out, d_in = M.shape
    Mg = M.reshape(d_out, d_in // m_group, m_group).astype(np.uint8)
    w = (1 << np.arange(m_group)).astype(np.uint8)
    return (Mg * w).sum(axis=2).astype(np.uint8)


def unpack_mask(Mb: np.ndarray, m_group: int = 4) -> np.ndarray:
    d_out, ng = Mb.shape
    bits = (Mb[:, :, None] >> np.arange(m_group)[None, None, :]) & 1
    return bits.astype(bool).reshape(d_out, ng * m_group)


# --------------------------------------------------------------------------
# O3  proxy loss (Eq. proxy_loss and its full-Gram generalisation)
# --------------------------------------------------------------------------
def residual(W, A, B, S):
    return np.asarray(W, dtype=np.float64) - bd_right(bd_left(A, S), B)


def proxy_loss(W, A, B, S, Hw) -> float:
    """L = sum_i e_i H_w e_i^T over the rows e_i of E = W - A S B."""
    E = residual(W, A, B, S)
    return float(np.sum((E @ Hw) * E))


# --------------------------------------------------------------------------
# O5  A-step: exact (proximal) minimiser of every row-block of A
# --------------------------------------------------------------------------
def a_step(W, A, B, S, Hw, cfg: OracleConfig):
    """With T = S B the loss of row-block i is tr((W_i - A_i T_i) H_w (.)^T),
    convex in A_i (Proposition 1).  Its gradient is -2 E_i H_w T_i^T (the
    gradient display of Appendix D.1); the step
        A_i += Gamma_i (G_i + lambda_i I)^-1,   G_i = T_i H_w T_i^T,
        Gamma_i = E_i H_w T_i^T,  lambda_i = ridge * tr(G_i) / d_block
    lands on its zero (ridge = 0) or on the proximal point.
    Reading: a block whose Cholesky fails is left unchanged."""
    db = cfg.d_block
    T = bd_right(S, B)
    E = np.asarray(W, dtype=np.float64) - bd_left(A, T)
    A = A.copy()
    failed = 0
    for i in range(A.shape[0]):
        r = slice(i * db, (i + 1) * db)
        Ti = T[r]
        G = Ti @ Hw @ Ti.T
        Gam = E[r] @ Hw @ Ti.T
        lam = cfg.ridge * np.trace(G) / db
        Gr = G + lam * np.eye(db)
        if not _is_spd(Gr):
            failed += 1
            continue
        A[i] = A[i] + np.linalg.solve(Gr, Gam.T).T
    return A, failed


def a_step_gd(W, A, B, S, Hw, cfg: OracleConfig):
    """The paper's own A update (Algorithm 2): one gradient step A <- A - eta_A grad_A L with the step of
    Eq. lrA, eta_A = 1 / beta_A, beta_A = 2 sum_{i,j} || T_ij D_j T_ij^T ||_F, T = (W' (.) M) B and D_j the
    j-th block of the diagonal weighting.  grad_{A_i} L = -2 E_i D T_i^T = -2 Gamma_i (Appendix D.1), so the move
    is Gamma_i / (beta_A / 2).  Defined for the diagonal weighting only, like the paper's loss."""
    db = cfg.d_block
    d = np.diag(Hw)
    T = bd_right(S, B)
    E = np.asarray(W, dtype=np.float64) - bd_left(A, T)
    nbo, nbi = A.shape[0], B.shape[0]
    half_beta = 0.0
    for i in range(nbo):
        for j in range(nbi):
            Tij = T[i * db:(i + 1) * db, j * db:(j + 1) * db]
            half_beta += np.linalg.norm((Tij * d[j * db:(j + 1) * db][None, :]) @ Tij.T)
    tau = 1.0 / half_beta if half_beta > 0.0 else 0.0
    A = A.copy()
    for i in range(nbo):
        r = slice(i * db, (i + 1) * db)
        A[i] = A[i] + tau * ((E[r] * d[None, :]) @ T[r].T)
    return A, tau


def b_step_gd(W, A, B, S, Hw, cfg: OracleConfig):
    """The paper's own B update: B <- B - eta_B grad_B L with Eq. lrB, eta_B = 1 / beta_B,
    beta_B = 2 sum_{i,j} || U_ij^T U_ij ||_F || D_j ||_F, U = A (W' (.) M) (Reading: S'^T S' for the printed
    S'^T S, as in the derivation above it).  grad_{B_j} L = -2 U_j^T (E D)_j = -2 Gamma_j (Appendix D.2)."""
    db = cfg.d_block
    d = np.diag(Hw)
    U = bd_left(A, S)
    E = np.asarray(W, dtype=np.float64) - bd_right(U, B)
    nbo, nbi = A.shape[0], B.shape[0]
    half_beta = 0.0
    for j in range(nbi):
        dn = np.linalg.norm(d[j * db:(j + 1) * db])
        for i in range(nbo):
            Uij = U[i * db:(i + 1) * db, j * db:(j + 1) * db]
            half_beta += np.linalg.norm(Uij.T @ Uij) * dn
    tau = 1.0 / half_beta if half_beta > 0.0 else 0.0
    B = B.copy()
    for j in range(nbi):
        c = slice(j * db, (j + 1) * db)
        B[j] = B[j] + tau * (U[:, c].T @ (E[:, c] * d[c][None, :]))
    return B, tau


def _is_spd(Mx: np.ndarray) -> bool:
    if not np.all(np.isfinite(Mx)):
        return False
    try:
        np.linalg.cholesky(Mx)
    except np.linalg.LinAlgError:
        return False
    return True


# --------------------------------------------------------------------------
# O6  B-step: simultaneous block-Newton directions, one exact scalar step
# --------------------------------------------------------------------------
def b_step(W, A, B, S, Hw, cfg: OracleConfig):
    """With U = A S the loss is tr((W - U B) H_w (W - U B)^T), convex in B.
    The negative half-gradient restricted to block j is
        Gamma_j = U_j^T (E H_w)_j          (Appendix D.2, with S'^T S' read
                                            for the printed S'^T S)
    and the block direction is
        Delta_j = (C_j + lambda_j I)^-1 Gamma_j (H_w,jj + mu_j I)^-1,
        C_j = U_j^T U_j.
    With diagonal weighting the column-blocks decouple (Eq. proxyBlock) and Delta_j is
    the exact minimiser, so tau = 1 up to the ridge.  Reading (full H_w): the
    blocks couple through off-diagonal blocks of H_w, so all blocks move along
    their Delta_j with one exact step
        tau = <Gamma, Delta> / tr(V H_w V^T),  V = U Delta,
    the monotone analogue of the paper's single global step size."""
    db = cfg.d_block
    U = bd_left(A, S)
    E = np.asarray(W, dtype=np.float64) - bd_right(U, B)
    EH = E @ Hw
    Delta = np.zeros_like(B)
    failed = 0
    gd = 0.0
    for j in range(B.shape[0]):
        c = slice(j * db, (j + 1) * db)
        Uj = U[:, c]
        C = Uj.T @ Uj
        Gam = Uj.T @ EH[:, c]
        Hjj = Hw[c, c]
        Cr = C + cfg.ridge * np.trace(C) / db * np.eye(db)
        Hr = Hjj + cfg.ridge * np.trace(Hjj) / db * np.eye(db)
        if not (_is_spd(Cr) and _is_spd(Hr)):
            failed += 1
            continue
        Y = np.linalg.solve(Cr, Gam)
        Delta[j] = np.linalg.solve(Hr, Y.T).T
        gd += float(np.sum(Gam * Delta[j]))
    V = bd_right(U, Delta)
    q = float(np.sum((V @ Hw) * V))
    tau = gd / q if q > 0.0 else 0.0
    return B + tau * Delta, tau, failed


# --------------------------------------------------------------------------
# O7  S-step: gradient step on the kept entries of the core
# --------------------------------------------------------------------------
def core_gradient(W, A, B, S, Hw):
    """Gamma = A^T E H_w B^T  (= -1/2 of the gradient display of Appendix D.3
    before the mask is applied)."""
    E = residual(W, A, B, S)
    return bd_left(bd_T(A), bd_right(E @ Hw, bd_T(B)))


def s_step(W, A, B, S, M, Hw, cfg: OracleConfig):
    """S += tau * (Gamma (.) M).  EXACT: tau minimises the loss along that
    direction, tau = ||Gamma_M||_F^2 / tr(V H_w V^T), V = A Gamma_M B.
    BETA: the paper's step 1/beta_W' (Eq. lrWprime): since the gradient is
    -2 Gamma_M, the move is Gamma_M / (||A^T A||_F ||B H_w B^T||_F)."""
    Gm = core_gradient(W, A, B, S, Hw) * M
    if cfg.s_step == S_BETA:
        AtA = np.einsum("bki,bkj->bij", A, A)
        Bd = bd_dense(B)
        beta_half = np.sqrt(np.sum(AtA * AtA)) * np.linalg.norm(Bd @ Hw @ Bd.T)
        tau = 1.0 / beta_half if beta_half > 0.0 else 0.0
    else:
        V = bd_right(bd_left(A, Gm), B)
        q = float(np.sum((V @ Hw) * V))
        tau = float(np.sum(Gm * Gm)) / q if q > 0.0 else 0.0
    return S + tau * Gm, tau


# --------------------------------------------------------------------------
# counter-based random numbers for the group selection
# --------------------------------------------------------------------------
_M64 = (1 << 64) - 1


def splitmix64(x: np.ndarray) -> np.ndarray:
    """The SplitMix64 output function on uint64 arrays (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        z = x.astype(np.uint64) + np.uint64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        return z ^ (z >> np.uint64(31))


def selection_uniform(seed: int, t: int, g: np.ndarray, n_groups_total: int) -> np.ndarray:
    """u_g in (0,1): (top 24 bits of splitmix64(seed ^ splitmix64(t*G + g)) + 0.5) / 2^24."""
    with np.errstate(over="ignore"):
        ctr = np.uint64(t & _M64) * np.uint64(n_groups_total) + g.astype(np.uint64)
        bits = splitmix64(np.uint64(seed & _M64) ^ splitmix64(ctr))
    return ((bits >> np.uint64(40)).astype(np.float64) + 0.5) * (2.0 ** -24)


# --------------------------------------------------------------------------
# O8  mask-step: the greedy sparse-core update (Algorithm 3, Appendix B.1)
# --------------------------------------------------------------------------
def pinv_solve(K: np.ndarray, z: np.ndarray):
    """(w, red) with w = K^+ z and red = z^T K^+ z for a small PSD K.
    2x2 (Eq. mask_loss_opt / mask_loss_opt_sol): Reading: if det <= 1e-12 K11 K22 use the rank-1
    pseudo-inverse K / tr(K)^2, and K^+ = 0 if tr K = 0.
    Larger n (N:M with n_keep > 2): Cholesky solve; returns None where the
    factorisation fails (that mask is skipped)."""
    n = K.shape[0]
    if n == 2:
        k11, k12, k22 = K[0, 0], K[0, 1], K[1, 1]
        det = k11 * k22 - k12 * k12
        if det <= 1e-12 * k11 * k22:
            tr = k11 + k22
            if tr <= 0.0:
                return np.zeros(2), 0.0
            w = (K @ z) / (tr * tr)
        else:
            w = np.array([k22 * z[0] - k12 * z[1], k11 * z[1] - k12 * z[0]]) / det
        return w, float(z @ w)
    if not _is_spd(K):
        return None
    w = np.linalg.solve(K, z)
    return w, float(z @ w)


def group_scores(Gamma: np.ndarray, m_group: int, select_mode: int = L1_RANDOM) -> np.ndarray:
    """l_g = L1 norm of the core gradient over all m positions of the group
    (Section 3.3.2).  Reading: masked-out positions count; their gradient is
    what signals a better mask.  The ablation of Appendix E.1 adds the L2 norm
    (L2_RANDOM) and equal weights (UNIFORM_RANDOM)."""
    d_out, d_in = Gamma.shape
    G = Gamma.reshape(d_out, d_in // m_group, m_group)
    if select_mode == L2_RANDOM:
        return np.sqrt((G * G).sum(axis=2))
    if select_mode == UNIFORM_RANDOM:
        return np.ones((d_out, d_in // m_group))
    return np.abs(G).sum(axis=2)


def mask_step(W, A, B, S, M, Hw, cfg: OracleConfig, t: int, info: IterInfo | None = None):
    """One group per (i, j) block is selected and re-solved over all masks.

    For the selected group (row r, columns m*c .. m*c+m-1), with a = A[:, r],
    alpha = ||a||^2, B_c the m rows of B of that group and K_c = B_c H_w B_c^T,
    freezing everything else gives (Appendix B.1)
        z = B_c H_w dW^T a = Gamma_g + alpha K_c s_g
    (dW = residual with the group's own contribution removed), and for a mask
    with kept positions P the best loss reduction and values are
        red_P = z_P^T K_PP^+ z_P / alpha,      w_P = K_PP^+ z_P / alpha
    (second term of Eq. mask_loss_opt; Eq. mask_loss_opt_sol).  Reading: the incumbent mask is evaluated
    first, then the others in lexicographic order, and a candidate replaces
    the best only on strict improvement, so ties keep the incumbent.
    Reading (full H_w): simultaneous updates in different column-blocks of one
    row-block interact, so all updates of the iteration are accepted only if
    the exact change of the loss, -2<E H_w, V> + tr(V H_w V^T) with
    V = A dS B, is <= 0, and discarded together otherwise.
    Reading (mask_groups = k > 1, not in the paper): the k groups with the smallest race keys are drawn in every
    block -- the exponential race then samples k groups without replacement with probability proportional to
    the score -- and each is re-solved on its own from the state before the update, exactly as a single group
    would be.  Groups of one block interact (they share columns of A or rows of B), so the test on the exact
    joint change of the loss above applies with either weighting."""
    db, n, m = cfg.d_block, cfg.n_keep, cfg.m_group
    kg = cfg.mask_groups
    d_out, d_in = S.shape
    nbo, nbi = d_out // db, d_in // db
    ng_row = d_in // m                      # groups per row
    gpb = db // m                           # groups per block row
    G_total = d_out * ng_row
    E = residual(W, A, B, S)
    EH = E @ Hw
    Gamma = bd_left(bd_T(A), bd_right(EH, bd_T(B)))
    alpha = np.einsum("bor,bor->br", A, A).reshape(d_out)          # ||A[:, r]||^2
    Kfull = np.stack([B[j] @ Hw[j * db:(j + 1) * db, j * db:(j + 1) * db] @ B[j].T
                      for j in range(nbi)])                        # [nbi, db, db]
    score = group_scores(Gamma, m, cfg.select_mode)                # [d_out, ng_row]
    score = np.where(alpha[:, None] > 0.0, score, 0.0)
    gidx = (np.arange(d_out, dtype=np.uint64)[:, None] * np.uint64(ng_row)
            + np.arange(ng_row, dtype=np.uint64)[None, :])
    if cfg.select_mode in (L1_RANDOM, L2_RANDOM, UNIFORM_RANDOM):
        u = selection_uniform(cfg.seed, t, gidx, G_total)
        with np.errstate(divide="ignore"):
            key = np.where(score > 0.0, -np.log(u) / score, np.inf)
    else:  # L1_GREEDY: arg-max of the score == arg-min of its negative
        key = np.where(score > 0.0, -score, np.inf)

    combos = list(itertools.combinations(range(m), n))
    dS = np.zeros_like(S)
    newM = M.copy()
    selected = -np.ones((nbo, nbi), dtype=np.int64)
    selected_all = -np.ones((nbo, nbi, kg), dtype=np.int64)
    sel_margin = np.full((nbo, nbi), np.inf)
    msk_margin = np.full((nbo, nbi), np.inf)
    new_mask = np.zeros((nbo, nbi), dtype=np.int64)
    def _solve_group(i, j, kk, p):
        r = i * db + p // gpb
        c = j * gpb + p % gpb           # group column index within the row
        if kk == 0:
            selected[i, j] = r * ng_row + c
        selected_all[i, j, kk] = r * ng_row + c
        cols = np.arange(m * c, m * c + m)
        lc = m * (p % gpb)              # group's first row inside B_j
        Kc = Kfull[j][lc:lc + m, lc:lc + m]
        a_r = alpha[r]
        s_g = S[r, cols]
        z = Gamma[r, cols] + a_r * (Kc @ s_g)
        inc = tuple(np.nonzero(M[r, cols])[0])
        order = [inc] + [cb for cb in combos if cb != inc]
        best = None
        reds = []
        for cb in order:
            ix = np.array(cb)
            sol = pinv_solve(Kc[np.ix_(ix, ix)], z[ix])
            if sol is None:
                continue
            w, red = sol
            red /= a_r
            reds.append(red)
            if best is None or red > best[0]:
                best = (red, cb, w / a_r)
        if best is None:
            return
        if len(reds) > 1:
            rs = np.sort(np.array(reds))[::-1]
            msk_margin[i, j] = min(msk_margin[i, j], (rs[0] - rs[1]) / max(abs(rs[0]), 1e-300))
        red, cb, w = best
        new_g = np.zeros(m)
        new_g[list(cb)] = w
        dS[r, cols] = new_g - s_g
        newM[r, cols] = False
        newM[r, m * c + np.array(cb)] = True
        if kk == 0:
            new_mask[i, j] = sum(1 << q for q in cb)

    for i in range(nbo):
        for j in range(nbi):
            kb = key[i * db:(i + 1) * db, j * gpb:(j + 1) * gpb]
            flat = kb.reshape(-1)           # row-major == ascending global group index
            picks = [int(q) for q in np.argsort(flat, kind="stable")[:kg] if np.isfinite(flat[q])]   # ties -> lowest g
            if not picks:
                continue
            if flat.size > len(picks) and len(picks) == kg:
                # how close the draw was: the gap between the last key taken and the first one left out
                srt = np.sort(flat)
                last_in, first_out = srt[kg - 1], srt[kg]
                if np.isfinite(first_out):
                    sel_margin[i, j] = abs(first_out - last_in) / max(abs(first_out), 1e-300)
            for kk, p in enumerate(picks):
                _solve_group(i, j, kk, p)
    V = bd_right(bd_left(A, dS), B)
    dL = float(-2.0 * np.sum(EH * V) + np.sum((V @ Hw) * V))
    accepted = dL <= 0.0
    if info is not None:
        info.selected, info.select_margin = selected, sel_margin
        info.selected_all = selected_all
        info.mask_margin, info.new_mask = msk_margin, new_mask
        info.delta_L_mask = dL
        info.mask_accepted = int(accepted)
        info.groups_changed = int(np.sum(np.any((newM != M).reshape(d_out, ng_row, m), axis=2))) if accepted else 0
    if not accepted:
        return S, M
    return S + dS, newM


# --------------------------------------------------------------------------
# O4  one BCD iteration and the outer loop (Algorithm 1)
# --------------------------------------------------------------------------
def adam_state(A, B, S):
    """First and second moment estimates of Adam for A, B and W', all zero."""
    return {k: np.zeros_like(x, dtype=np.float64) for k, x in
            (("mA", A), ("vA", A), ("mB", B), ("vB", B), ("mS", S), ("vS", S))}


def joint_gradients(W, A, B, S, M, Hw, cfg: OracleConfig):
    """Gradients of the loss with respect to A, B and W' at one and the same point (Appendix D.1-D.3):
    -2 E_i H_w T_i^T, -2 U_j^T (E H_w)_j and -2 (A^T E H_w B^T) (.) M."""
    db = cfg.d_block
    T = bd_right(S, B)
    U = bd_left(A, S)
    E = np.asarray(W, dtype=np.float64) - bd_left(A, T)
    EH = E @ Hw
    gA = np.stack([-2.0 * EH[i * db:(i + 1) * db] @ T[i * db:(i + 1) * db].T for i in range(A.shape[0])])
    gB = np.stack([-2.0 * U[:, j * db:(j + 1) * db].T @ EH[:, j * db:(j + 1) * db] for j in range(B.shape[0])])
    gS = -2.0 * bd_left(bd_T(A), bd_right(EH, bd_T(B))) * M
    return gA, gB, gS


def adam_joint_step(W, A, B, S, M, Hw, cfg: OracleConfig, state: dict, t_adam: int):
    """What the paper runs in practice (Section 3.3.1): one Adam step (Kingma & Ba, Algorithm 1 with bias
    correction) on A, B and W' together, from gradients taken at the same point.  t_adam counts from 1.
    The state dict is updated in place."""
    b1, b2, lr, eps = cfg.adam_beta1, cfg.adam_beta2, cfg.adam_lr, cfg.adam_eps
    grads = dict(zip("ABS", joint_gradients(W, A, B, S, M, Hw, cfg)))
    new = {}
    for k, theta in (("A", A), ("B", B), ("S", S)):
        g = grads[k]
        m = state["m" + k] = b1 * state["m" + k] + (1.0 - b1) * g
        v = state["v" + k] = b2 * state["v" + k] + (1.0 - b2) * g * g
        mhat = m / (1.0 - b1 ** t_adam)
        vhat = v / (1.0 - b2 ** t_adam)
        new[k] = theta - lr * mhat / (np.sqrt(vhat) + eps)
    # Reading: the core is W' (.) M, so an entry that the sparse-core update has masked out stays zero even while
    # its first moment is still decaying; the moments themselves are left alone when a mask changes.
    return new["A"], new["B"], new["S"] * M


def mask_phase(W, A, B, S, M, Hw, cfg: OracleConfig, t: int, info: IterInfo):
    """The sparse-core update of iteration t: Algorithm 3 run cfg.mask_sweeps times in a row, each run from
    the state the previous one left (fresh residual, fresh gradient, fresh selection).
    Reading: the paper alternates one continuous and one sparse-core update; with mask_sweeps = K the loop is
    the same alternation with the continuous update skipped on K-1 of every K turns, so run k of iteration t
    draws its selection with the counter t*K + k (for K = 1 this is t).  Each run keeps Lemma 2's guarantee,
    so the loss cannot rise across the phase.  The record sums the loss changes evaluated, the runs accepted
    and the groups changed; the selection fields are those of the last run."""
    K = cfg.mask_sweeps
    info.mask_accepted, info.delta_L_mask, info.groups_changed = 0, 0.0, 0
    for k in range(K):
        sub = IterInfo()
        S, M = mask_step(W, A, B, S, M, Hw, cfg, t * K + k, sub)
        info.sweeps.append(sub)
        info.mask_accepted += sub.mask_accepted
        info.delta_L_mask += sub.delta_L_mask
        info.groups_changed += sub.groups_changed
    last = info.sweeps[-1]
    info.selected, info.select_margin = last.selected, last.select_margin
    info.mask_margin, info.new_mask = last.mask_margin, last.new_mask
    return S, M


def bcd_iteration(W, A, B, S, M, Hw, cfg: OracleConfig, t: int, want_loss: bool = True, opt_state: dict | None = None):
    """A-step, then B-step with the new A, then S-step with the new A and B
    (the order of Algorithm 2 / Lemma 1), then the sparse-core update
    (Algorithm 3).  Every sub-step recomputes the residual from scratch."""
    info = IterInfo()
    if want_loss:
        info.loss["start"] = proxy_loss(W, A, B, S, Hw)
    if cfg.ab_step == AB_GD and cfg.h_mode != DIAG:
        raise ValueError("the paper's gradient steps for A and B are defined for the diagonal weighting")
    if cfg.ab_step == AB_ADAM:
        # joint Adam replaces the three sequential sub-steps; then the sparse-core update as usual
        if opt_state is None:
            raise ValueError("joint Adam needs its moment estimates (adam_state)")
        A, B, S = adam_joint_step(W, A, B, S, M, Hw, cfg, opt_state, t + 1)
        if want_loss:
            info.loss["A"] = info.loss["B"] = info.loss["S"] = proxy_loss(W, A, B, S, Hw)
        if cfg.phases & PH_MASK:
            S, M = mask_phase(W, A, B, S, M, Hw, cfg, t, info)
            if want_loss:
                info.loss["mask"] = proxy_loss(W, A, B, S, Hw)
        return A, B, S, M, info
    if cfg.phases & PH_A:
        if cfg.ab_step == AB_GD:
            A, info.tau_A = a_step_gd(W, A, B, S, Hw, cfg)
        else:
            A, f = a_step(W, A, B, S, Hw, cfg)
            info.chol_failed += f
        if want_loss:
            info.loss["A"] = proxy_loss(W, A, B, S, Hw)
    if cfg.phases & PH_B:
        if cfg.ab_step == AB_GD:
            B, info.tau_B = b_step_gd(W, A, B, S, Hw, cfg)
        else:
            B, info.tau_B, f = b_step(W, A, B, S, Hw, cfg)
            info.chol_failed += f
        if want_loss:
            info.loss["B"] = proxy_loss(W, A, B, S, Hw)
    if cfg.phases & PH_S:
        S, info.tau_S = s_step(W, A, B, S, M, Hw, cfg)
        if want_loss:
            info.loss["S"] = proxy_loss(W, A, B, S, Hw)
    if cfg.phases & PH_MASK:
        S, M = mask_phase(W, A, B, S, M, Hw, cfg, t, info)
        if want_loss:
            info.loss["mask"] = proxy_loss(W, A, B, S, Hw)
    return A, B, S, M, info


def run(W, H, cfg: OracleConfig, n_iters: int, t_first: int = 0, state=None, want_loss: bool = True,
        opt_state: dict | None = None):
    """Algorithm 1 without the normalisation (apply normalize() first if wanted).
    Returns the final (A, B, S, M) and the per-iteration IterInfo list."""
    Hw = weighting(H, cfg.h_mode)
    W = np.asarray(W, dtype=np.float64)
    if state is None:
        A, B, S, M = init(W, H, cfg)
    else:
        A, B, S, M = (np.array(x) for x in state)
    infos = []
    if cfg.ab_step == AB_ADAM and opt_state is None:
        opt_state = adam_state(A, B, S)
    for k in range(n_iters):
        A, B, S, M, info = bcd_iteration(W, A, B, S, M, Hw, cfg, t_first + k, want_loss, opt_state)
        infos.append(info)
    return (A, B, S, M), infos


# --------------------------------------------------------------------------
# deployment form (Section 3.1, Section 3.2 last paragraph)
# --------------------------------------------------------------------------
def apply(A, B, S, x, r1=None, r2=None) -> np.ndarray:
    """y_t = A (S (B x_t)) for every row x_t of x [n_tokens, d_in].
    With r1, r2: y_t = diag(r2) A S B diag(r1) x_t, i.e. the normalisation is
    undone by scaling B's columns by r1 and A's rows by r2 (the pairing the
    dimensions force)."""
    x = np.asarray(x, dtype=np.float64)
    if r1 is not None:
        x = x * r1[None, :]
    z1 = bd_right(x, bd_T(B))            # (B x)^T  = x^T B^T
    z2 = z1 @ S.T
    y = bd_right(z2, bd_T(A))
    if r2 is not None:
        y = y * r2[None, :]
    return y


def overhead_fraction(d_out: int, d_in: int, d_block: int) -> float:
    """Extra parameters of the wrappers relative to the dense layer (Section 3.1)."""
    return (d_out + d_in) * d_block / (d_out * d_in)
