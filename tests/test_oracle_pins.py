"""Pins for the CPU oracle: every function is checked against something other
than itself -- a definition written out with loops, textbook least squares on
the vectorised problem, brute force, finite differences, a closed form, or a
theorem of the paper.  No GPU is involved."""
import itertools
import os

import numpy as np
import pytest

from oracle import armor_oracle as O
from paper_2510_05528_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def tiny(d_out=16, d_in=24, db=8, n=96, seed=0, outliers=2):
    cfg = inputs.LayerConfig("t", d_out, d_in, db, n, 4, seed=seed, n_outlier=outliers,
                             outlier_scale=20.0, chunk_rows=32)
    W = inputs.make_weight(cfg).astype(np.float64)
    X = inputs.make_activations(cfg).astype(np.float64)
    return cfg, W, X


def rand_state(W, H, ocfg, rng, scale=0.1):
    """A perturbed state: wrappers away from identity, core values away from W."""
    A, B, S, M = O.init(W, H, ocfg)
    A = A + scale * rng.standard_normal(A.shape)
    B = B + scale * rng.standard_normal(B.shape)
    S = (S + scale * 0.02 * rng.standard_normal(S.shape)) * M
    return A, B, S, M


def loss_from_X(W, A, B, S, X):
    """tr(E H E^T) = ||E X^T||_F^2 straight from the activations (no Gram)."""
    E = W - O.bd_dense(A) @ S @ O.bd_dense(B)
    return float(np.linalg.norm(E @ X.T) ** 2)


# ------------------------------------------------------------------ Gram, loss
def test_gram_is_sum_of_outer_products():
    _, _, X = tiny(n=40)
    H = O.gram(X)
    ref = np.zeros_like(H)
    for t in range(X.shape[0]):
        ref += np.outer(X[t], X[t])
    assert np.allclose(H, ref, rtol=1e-12, atol=1e-9)
    assert np.allclose(H, H.T)
    assert np.allclose(np.diag(H), (X ** 2).sum(axis=0))
    # accumulation over chunks
    H2 = O.gram(X[20:], O.gram(X[:20]))
    assert np.allclose(H, H2, rtol=1e-12)


def test_full_loss_equals_norm_of_E_Xt():
    cfg, W, X = tiny()
    H = O.gram(X)
    oc = O.OracleConfig(cfg.d_block)
    A, B, S, M = rand_state(W, H, oc, np.random.default_rng(1))
    assert np.isclose(O.proxy_loss(W, A, B, S, O.weighting(H, O.FULL)),
                      loss_from_X(W, A, B, S, X), rtol=1e-10)


def test_diag_loss_is_the_papers_double_sum_and_block_sum():
    cfg, W, X = tiny()
    H = O.gram(X)
    db = cfg.d_block
    oc = O.OracleConfig(db, h_mode=O.DIAG)
    A, B, S, M = rand_state(W, H, oc, np.random.default_rng(2))
    What = O.bd_dense(A) @ S @ O.bd_dense(B)
    xn = (X ** 2).sum(axis=0)
    dbl = 0.0
    for i in range(W.shape[0]):
        for j in range(W.shape[1]):
            dbl += (W[i, j] - What[i, j]) ** 2 * xn[j]
    L = O.proxy_loss(W, A, B, S, O.weighting(H, O.DIAG))
    assert np.isclose(L, dbl, rtol=1e-10)
    # Eq. proxyBlock: sum over (i, j) blocks of the block's own weighted norm
    blk = 0.0
    for i in range(W.shape[0] // db):
        for j in range(W.shape[1] // db):
            r, c = slice(i * db, (i + 1) * db), slice(j * db, (j + 1) * db)
            Eb = W[r, c] - A[i] @ S[r, c] @ B[j]
            blk += np.sum(Eb ** 2 * xn[c][None, :])
    assert np.isclose(L, blk, rtol=1e-10)
    assert L >= 0.0


# ------------------------------------------------------------------ normalise
def test_normalize_formulas_and_unit_rows():
    _, W, _ = tiny()
    Wb, r1, r2 = O.normalize(W)
    for j in range(W.shape[1]):
        assert np.isclose(r1[j], np.sqrt(sum(W[i, j] ** 2 for i in range(W.shape[0]))))
    for i in range(W.shape[0]):
        assert np.isclose(r2[i], np.sqrt(sum((W[i, j] / r1[j]) ** 2 for j in range(W.shape[1]))))
    assert np.allclose(Wb * r2[:, None] * r1[None, :], W)
    assert np.allclose((Wb ** 2).sum(axis=1), 1.0)
    assert np.isclose((Wb ** 2).sum(), W.shape[0])
    W0 = W.copy()
    W0[:, 3] = 0.0
    W0[5, :] = 0.0
    Wb0, r10, r20 = O.normalize(W0)
    assert r10[3] == 1.0 and r20[5] == 1.0 and np.all(np.isfinite(Wb0))


# ------------------------------------------------------------------ init
def test_init_is_optimal_for_identity_wrappers_by_brute_force():
    cfg, W, X = tiny(d_out=8, d_in=16, db=8)
    H = O.gram(X)
    oc = O.OracleConfig(cfg.d_block, h_mode=O.DIAG)
    A, B, S, M = O.init(W, H, oc)
    assert np.all(A == np.eye(8)[None]) and np.all(B == np.eye(8)[None])
    assert np.all(M.reshape(8, 4, 4).sum(axis=2) == 2)
    assert np.all(S == W * M)
    d = np.diag(H)
    # brute force: with A = B = I the loss separates per group; for a mask the best
    # values are W on the kept entries, so the group loss is the pruned W^2 d.
    for i in range(8):
        for c in range(4):
            cols = np.arange(4 * c, 4 * c + 4)
            losses = {}
            for keep in itertools.combinations(range(4), 2):
                drop = [p for p in range(4) if p not in keep]
                losses[keep] = sum(W[i, cols[p]] ** 2 * d[cols[p]] for p in drop)
            best = min(losses, key=losses.get)
            assert tuple(np.nonzero(M[i, cols])[0]) == best
    closed = np.sum((W ** 2 * d[None, :])[~M])
    assert np.isclose(O.proxy_loss(W, A, B, S, O.weighting(H, O.DIAG)), closed, rtol=1e-12)


def test_init_ties_keep_lower_index_and_pack_roundtrip():
    W = np.ones((2, 8))
    H = np.eye(8)
    _, _, _, M = O.init(W, H, O.OracleConfig(4))
    assert np.all(M == np.array([1, 1, 0, 0, 1, 1, 0, 0], dtype=bool)[None, :])
    Mb = O.pack_mask(M)
    assert Mb.dtype == np.uint8 and np.all(Mb == 3)
    rng = np.random.default_rng(0)
    Mr = rng.random((4, 16)) < 0.5
    assert np.all(O.unpack_mask(O.pack_mask(Mr)) == Mr)
    _, _, _, M48 = O.init(rng.standard_normal((4, 16)), np.eye(16), O.OracleConfig(8, n_keep=4, m_group=8))
    assert np.all(M48.reshape(4, 2, 8).sum(axis=2) == 4)
    for n_keep in (5, 6):     # the denser patterns of Section 4.4: the n largest |w| of every eight (H = I)
        Wn = rng.standard_normal((4, 16))
        _, _, _, Mn = O.init(Wn, np.eye(16), O.OracleConfig(8, n_keep=n_keep, m_group=8))
        kept = np.sort(np.abs(Wn).reshape(4, 2, 8), axis=2)[:, :, 8 - n_keep:]
        assert np.array_equal(np.sort(np.abs(Wn * Mn).reshape(4, 2, 8), axis=2)[:, :, 8 - n_keep:], kept)
        assert np.all(Mn.reshape(4, 2, 8).sum(axis=2) == n_keep)


# ------------------------------------------------------------------ A-step
@pytest.mark.parametrize("h_mode", [O.FULL, O.DIAG])
def test_a_step_is_the_least_squares_solution(h_mode):
    cfg, W, X = tiny()
    H = O.gram(X)
    db = cfg.d_block
    oc = O.OracleConfig(db, h_mode=h_mode, ridge=0.0)
    Hw = O.weighting(H, h_mode)
    A, B, S, M = rand_state(W, H, oc, np.random.default_rng(3))
    A1, failed = O.a_step(W, A, B, S, Hw, oc)
    assert failed == 0
    # textbook: min_Ai || (W_i - A_i T_i) R ||_F with R R^T = H_w
    R = X.T if h_mode == O.FULL else np.diag(np.sqrt(np.diag(H)))
    T = S @ O.bd_dense(B)
    for i in range(A.shape[0]):
        r = slice(i * db, (i + 1) * db)
        sol, *_ = np.linalg.lstsq((T[r] @ R).T, (W[r] @ R).T, rcond=None)
        assert np.allclose(A1[i], sol.T, rtol=1e-6, atol=1e-8)
    # the paper's gradient (Appendix D.1), summed over j, vanishes at the new A (DIAG)
    if h_mode == O.DIAG:
        d = np.diag(H)
        for i in range(A.shape[0]):
            g = np.zeros((db, db))
            for j in range(B.shape[0]):
                r, c = slice(i * db, (i + 1) * db), slice(j * db, (j + 1) * db)
                Sij = S[r, c] @ B[j]
                D = np.diag(d[c])
                g += 2 * A1[i] @ (Sij @ D @ Sij.T) - 2 * W[r, c] @ D @ Sij.T
            assert np.linalg.norm(g) < 1e-8 * np.linalg.norm(W) * d.max()
    assert O.proxy_loss(W, A1, B, S, Hw) <= O.proxy_loss(W, A, B, S, Hw)


def test_a_step_ridge_is_proximal_and_singular_block_is_skipped():
    cfg, W, X = tiny()
    H = O.gram(X)
    oc = O.OracleConfig(cfg.d_block, ridge=1e-3)
    Hw = O.weighting(H, O.FULL)
    A, B, S, M = rand_state(W, H, oc, np.random.default_rng(4))
    L0 = O.proxy_loss(W, A, B, S, Hw)
    A1, _ = O.a_step(W, A, B, S, Hw, oc)
    assert O.proxy_loss(W, A1, B, S, Hw) <= L0
    S0 = S.copy()
    S0[: cfg.d_block] = 0.0                       # T_0 = 0 -> G_0 = 0: not SPD even with the ridge
    A2, failed = O.a_step(W, A, B, S0, Hw, oc)
    assert failed == 1 and np.all(A2[0] == A[0])


# ------------------------------------------------------------------ B-step
def test_b_step_diag_is_the_least_squares_solution():
    cfg, W, X = tiny()
    H = O.gram(X)
    db = cfg.d_block
    oc = O.OracleConfig(db, h_mode=O.DIAG, ridge=0.0)
    Hw = O.weighting(H, O.DIAG)
    A, B, S, M = rand_state(W, H, oc, np.random.default_rng(5))
    B1, tau, failed = O.b_step(W, A, B, S, Hw, oc)
    assert failed == 0 and np.isclose(tau, 1.0, rtol=1e-9)
    U = O.bd_dense(A) @ S
    d = np.diag(H)
    for j in range(B.shape[0]):
        c = slice(j * db, (j + 1) * db)
        # every column of W_j is fitted separately by U_j b (weights d_c > 0 cancel)
        sol, *_ = np.linalg.lstsq(U[:, c], W[:, c], rcond=None)
        assert np.allclose(B1[j], sol, rtol=1e-6, atol=1e-9)
        # the derived gradient 2 U_j^T U_j B_j D - 2 U_j^T W_j D vanishes
        D = np.diag(d[c])
        g = 2 * U[:, c].T @ U[:, c] @ B1[j] @ D - 2 * U[:, c].T @ W[:, c] @ D
        assert np.linalg.norm(g) < 1e-8 * d.max()


@pytest.mark.parametrize("h_mode", [O.FULL, O.DIAG])
def test_b_step_decrease_is_the_closed_form_of_a_1d_quadratic(h_mode):
    cfg, W, X = tiny()
    H = O.gram(X)
    db = cfg.d_block
    oc = O.OracleConfig(db, h_mode=h_mode)
    Hw = O.weighting(H, h_mode)
    A, B, S, M = rand_state(W, H, oc, np.random.default_rng(6))
    L0 = O.proxy_loss(W, A, B, S, Hw)
    B1, tau, _ = O.b_step(W, A, B, S, Hw, oc)
    L1 = O.proxy_loss(W, A, B1, S, Hw)
    Delta = (B1 - B) / tau
    # directional derivative by central differences and curvature by second difference
    eps = 1e-4
    f = lambda s: O.proxy_loss(W, A, B + s * Delta, S, Hw)
    slope = (f(eps) - f(-eps)) / (2 * eps)
    curv = (f(eps) - 2 * L0 + f(-eps)) / eps ** 2
    assert np.isclose(tau, -slope / curv, rtol=1e-5)
    assert np.isclose(L0 - L1, slope ** 2 / (2 * curv), rtol=1e-5)
    assert L1 <= L0
    # a line search cannot be improved by a small extra move along the same direction
    assert f(tau) <= min(f(tau * 1.01), f(tau * 0.99))


def test_b_direction_is_minus_half_gradient_preconditioned():
    """Gamma_j equals -1/2 dL/dB_j by finite differences (pins the S'^T S' reading)."""
    cfg, W, X = tiny(d_out=8, d_in=8, db=4, n=40)
    H = O.gram(X)
    oc = O.OracleConfig(4, ridge=0.0)
    Hw = O.weighting(H, O.FULL)
    A, B, S, M = rand_state(W, H, oc, np.random.default_rng(7))
    U = O.bd_dense(A) @ S
    EH = (W - U @ O.bd_dense(B)) @ Hw
    eps = 1e-6
    for j in range(2):
        c = slice(4 * j, 4 * j + 4)
        Gam = U[:, c].T @ EH[:, c]
        num = np.zeros((4, 4))
        for a in range(4):
            for b in range(4):
                Bp, Bm = B.copy(), B.copy()
                Bp[j, a, b] += eps
                Bm[j, a, b] -= eps
                num[a, b] = (O.proxy_loss(W, A, Bp, S, Hw) - O.proxy_loss(W, A, Bm, S, Hw)) / (2 * eps)
        assert np.allclose(-0.5 * num, Gam, rtol=1e-5, atol=1e-7 * np.abs(Gam).max())


# ------------------------------------------------------------------ S-step
@pytest.mark.parametrize("h_mode", [O.FULL, O.DIAG])
def test_core_gradient_matches_finite_differences_and_paper_formula(h_mode):
    cfg, W, X = tiny(d_out=8, d_in=8, db=4, n=40)
    H = O.gram(X)
    oc = O.OracleConfig(4, h_mode=h_mode)
    Hw = O.weighting(H, h_mode)
    A, B, S, M = rand_state(W, H, oc, np.random.default_rng(8))
    Gamma = O.core_gradient(W, A, B, S, Hw)
    eps = 1e-6
    num = np.zeros_like(S)
    for i in range(8):
        for j in range(8):
            Sp, Sm = S.copy(), S.copy()
            Sp[i, j] += eps
            Sm[i, j] -= eps
            num[i, j] = (O.proxy_loss(W, A, B, Sp, Hw) - O.proxy_loss(W, A, B, Sm, Hw)) / (2 * eps)
    assert np.allclose(-0.5 * num, Gamma, rtol=1e-5, atol=1e-7 * np.abs(Gamma).max())
    if h_mode == O.DIAG:      # the display of Appendix D.3
        Ad, Bd, D = O.bd_dense(A), O.bd_dense(B), np.diag(np.diag(H))
        grad = (2 * Ad.T @ Ad @ S @ Bd @ D @ Bd.T - 2 * Ad.T @ W @ D @ Bd.T) * M
        assert np.allclose(grad, -2 * Gamma * M, rtol=1e-9, atol=1e-12)


@pytest.mark.parametrize("h_mode", [O.FULL, O.DIAG])
def test_s_step_exact_decrease_and_beta_step(h_mode):
    cfg, W, X = tiny()
    H = O.gram(X)
    oc = O.OracleConfig(cfg.d_block, h_mode=h_mode)
    Hw = O.weighting(H, h_mode)
    A, B, S, M = rand_state(W, H, oc, np.random.default_rng(9))
    L0 = O.proxy_loss(W, A, B, S, Hw)
    Gm = O.core_gradient(W, A, B, S, Hw) * M
    S1, tau = O.s_step(W, A, B, S, M, Hw, oc)
    assert np.all(S1[~M] == 0.0)
    V = O.bd_dense(A) @ Gm @ O.bd_dense(B)
    q = np.linalg.norm(V @ X.T) ** 2 if h_mode == O.FULL else np.sum(V ** 2 * np.diag(H)[None, :])
    assert np.isclose(tau, np.sum(Gm ** 2) / q, rtol=1e-9)
    assert np.isclose(L0 - O.proxy_loss(W, A, B, S1, Hw), np.sum(Gm ** 2) ** 2 / q, rtol=1e-6)
    # BETA: step 1/beta with beta = 2 ||A^T A||_F ||B H_w B^T||_F; monotone by smoothness
    ob = O.OracleConfig(cfg.d_block, h_mode=h_mode, s_step=O.S_BETA)
    S2, tb = O.s_step(W, A, B, S, M, Hw, ob)
    Ad, Bd = O.bd_dense(A), O.bd_dense(B)
    beta = 2 * np.linalg.norm(Ad.T @ Ad) * np.linalg.norm(Bd @ Hw @ Bd.T)
    assert np.isclose(tb, 2.0 / beta, rtol=1e-12)
    assert np.allclose(S2, S - (1.0 / beta) * (-2 * Gm))
    L2 = O.proxy_loss(W, A, B, S2, Hw)
    assert L2 <= L0 and L2 >= O.proxy_loss(W, A, B, S1, Hw) - 1e-12 * L0


# ------------------------------------------------------------------ group solve
@pytest.mark.parametrize("h_mode", [O.FULL, O.DIAG])
def test_group_solve_matches_brute_force_least_squares(h_mode):
    """For every group and each of the 6 masks: fit the two free values by generic
    least squares on the full loss and compare values and loss with the closed form."""
    cfg, W, X = tiny(d_out=8, d_in=8, db=4, n=40)
    H = O.gram(X)
    Hw = O.weighting(H, h_mode)
    R = X.T if h_mode == O.FULL else np.diag(np.sqrt(np.diag(H)))
    oc = O.OracleConfig(4, h_mode=h_mode)
    A, B, S, M = rand_state(W, H, oc, np.random.default_rng(10), scale=0.3)
    Ad, Bd = O.bd_dense(A), O.bd_dense(B)
    Gamma = O.core_gradient(W, A, B, S, Hw)
    L0 = O.proxy_loss(W, A, B, S, Hw)
    for r, c in [(0, 0), (3, 1), (5, 0), (7, 1)]:
        cols = np.arange(4 * c, 4 * c + 4)
        S0 = S.copy()
        S0[r, cols] = 0.0
        dW = W - Ad @ S0 @ Bd
        Lfrozen = np.linalg.norm(dW @ R) ** 2
        a = Ad[:, r]
        alpha = a @ a
        Kc = Bd[cols] @ Hw @ Bd[cols].T
        z = Gamma[r, cols] + alpha * Kc @ S[r, cols]
        assert np.allclose(z, Bd[cols] @ Hw @ dW.T @ a, rtol=1e-9, atol=1e-12)
        for keep in itertools.combinations(range(4), 2):
            ix = np.array(keep)
            # vec(a w^T B') is linear in w: columns of the design matrix
            cols_design = [np.outer(a, Bd[cols[p]]) @ R for p in keep]
            Dm = np.stack([m.reshape(-1) for m in cols_design], axis=1)
            sol, *_ = np.linalg.lstsq(Dm, (dW @ R).reshape(-1), rcond=None)
            Lbest = np.linalg.norm((dW @ R).reshape(-1) - Dm @ sol) ** 2
            w, red = O.pinv_solve(Kc[np.ix_(ix, ix)], z[ix])
            assert np.allclose(w / alpha, sol, rtol=1e-7, atol=1e-10)
            assert np.isclose(Lfrozen - red / alpha, Lbest, rtol=1e-9, atol=1e-12 * L0)


@pytest.mark.parametrize("n_keep", [4, 5, 6])
@pytest.mark.parametrize("h_mode", [O.FULL, O.DIAG])
def test_group_solve_n_of_8_matches_brute_force_least_squares(h_mode, n_keep):
    """The 4:8, 5:8 and 6:8 patterns (Section 4.4): for a group and each of its 70 / 56 / 28 masks the free
    values fitted by generic least squares on the full loss agree with the closed form, and the mask step's
    choice is the best of all masks."""
    cfg, W, X = tiny(d_out=8, d_in=16, db=8, n=60)
    H = O.gram(X)
    Hw = O.weighting(H, h_mode)
    R = X.T if h_mode == O.FULL else np.diag(np.sqrt(np.diag(H)))
    oc = O.OracleConfig(8, n_keep=n_keep, m_group=8, h_mode=h_mode, select_mode=O.L1_GREEDY, phases=O.PH_MASK)
    A, B, S, M = rand_state(W, H, oc, np.random.default_rng(12), scale=0.3)
    assert np.all(M.reshape(8, -1, 8).sum(axis=2) == n_keep)
    Ad, Bd = O.bd_dense(A), O.bd_dense(B)
    Gamma = O.core_gradient(W, A, B, S, Hw)
    r, c = 5, 1
    cols = np.arange(8 * c, 8 * c + 8)
    S0 = S.copy()
    S0[r, cols] = 0.0
    dW = W - Ad @ S0 @ Bd
    Lfrozen = np.linalg.norm(dW @ R) ** 2
    a = Ad[:, r]
    alpha = a @ a
    Kc = Bd[cols] @ Hw @ Bd[cols].T
    z = Gamma[r, cols] + alpha * Kc @ S[r, cols]
    combos = list(itertools.combinations(range(8), n_keep))
    assert len(combos) == {4: 70, 5: 56, 6: 28}[n_keep]
    for keep in combos[::7] + [combos[-1]]:
        ix = np.array(keep)
        Dm = np.stack([(np.outer(a, Bd[cols[p]]) @ R).reshape(-1) for p in keep], axis=1)
        sol, *_ = np.linalg.lstsq(Dm, (dW @ R).reshape(-1), rcond=None)
        Lbest = np.linalg.norm((dW @ R).reshape(-1) - Dm @ sol) ** 2
        w, red = O.pinv_solve(Kc[np.ix_(ix, ix)], z[ix])
        assert np.allclose(w / alpha, sol, rtol=1e-6, atol=1e-10)
        assert np.isclose(Lfrozen - red / alpha, Lbest, rtol=1e-8)
    # the whole mask step with one block: greedy selection, best of the 70 masks, loss cannot rise
    info = O.IterInfo()
    L0 = O.proxy_loss(W, A, B, S, Hw)
    S1, M1 = O.mask_step(W, A, B, S, M, Hw, oc, 0, info)
    assert np.all(M1.reshape(8, -1, 8).sum(axis=2) == n_keep) and np.all(S1[~M1] == 0.0)
    assert O.proxy_loss(W, A, B, S1, Hw) <= L0 * (1 + 1e-12)
    for j in range(2):
        g = int(info.selected[0, j])
        rr, cc = divmod(g, 2)
        cs = np.arange(8 * cc, 8 * cc + 8)
        S0 = S.copy()
        S0[rr, cs] = 0.0
        dWj = (W - Ad @ S0 @ Bd) @ R
        best = (np.inf, None)
        for keep in combos:
            Dm = np.stack([(np.outer(Ad[:, rr], Bd[cs[p]]) @ R).reshape(-1) for p in keep], axis=1)
            sol, *_ = np.linalg.lstsq(Dm, dWj.reshape(-1), rcond=None)
            Lm = np.linalg.norm(dWj.reshape(-1) - Dm @ sol) ** 2
            if Lm < best[0] * (1 - 1e-12):
                best = (Lm, keep)
        if info.mask_accepted and info.mask_margin[0, j] > 1e-9:
            assert tuple(np.nonzero(M1[rr, cs])[0]) == best[1]


def test_pinv_solve_singular_cases():
    v = np.array([1.0, 2.0])
    K = np.outer(v, v)
    z = np.array([0.5, -0.3])
    w, red = O.pinv_solve(K, z)
    assert np.allclose(w, np.linalg.pinv(K) @ z) and np.isclose(red, z @ np.linalg.pinv(K) @ z)
    w0, r0 = O.pinv_solve(np.zeros((2, 2)), z)
    assert np.all(w0 == 0) and r0 == 0.0
    K4 = np.eye(4) + 0.1
    z4 = np.arange(4.0)
    w4, r4 = O.pinv_solve(K4, z4)
    assert np.allclose(K4 @ w4, z4) and np.isclose(r4, z4 @ w4)
    assert O.pinv_solve(np.zeros((4, 4)), z4) is None


# ------------------------------------------------------------------ mask step
def test_mask_step_is_a_fixed_point_at_init_in_diag_mode():
    cfg, W, X = tiny()
    H = O.gram(X)
    oc = O.OracleConfig(cfg.d_block, h_mode=O.DIAG, phases=O.PH_MASK)
    Hw = O.weighting(H, O.DIAG)
    A, B, S, M = O.init(W, H, oc)
    info = O.IterInfo()
    S1, M1 = O.mask_step(W, A, B, S, M, Hw, oc, 0, info)
    assert np.all(M1 == M) and np.allclose(S1, S, rtol=1e-12, atol=1e-15)
    assert info.groups_changed == 0 and np.all(info.selected >= 0)


@pytest.mark.parametrize("h_mode,select", [(O.DIAG, O.L1_RANDOM), (O.DIAG, O.L1_GREEDY),
                                           (O.FULL, O.L1_RANDOM), (O.FULL, O.L1_GREEDY)])
def test_mask_step_picks_the_brute_force_optimum_for_each_selected_group(h_mode, select):
    cfg, W, X = tiny()
    H = O.gram(X)
    db = cfg.d_block
    Hw = O.weighting(H, h_mode)
    R = X.T if h_mode == O.FULL else np.diag(np.sqrt(np.diag(H)))
    oc = O.OracleConfig(db, h_mode=h_mode, select_mode=select, seed=5)
    A, B, S, M = rand_state(W, H, oc, np.random.default_rng(11), scale=0.2)
    info = O.IterInfo()
    L0 = O.proxy_loss(W, A, B, S, Hw)
    S1, M1 = O.mask_step(W, A, B, S, M, Hw, oc, 3, info)
    assert np.all(M1.reshape(W.shape[0], -1, 4).sum(axis=2) == 2)
    assert np.all(S1[~M1] == 0.0)
    L1 = O.proxy_loss(W, A, B, S1, Hw)
    assert L1 <= L0 * (1 + 1e-12)
    if h_mode == O.DIAG:
        assert info.mask_accepted == 1
    if not info.mask_accepted:
        assert np.all(S1 == S) and np.all(M1 == M)
        return
    Ad, Bd = O.bd_dense(A), O.bd_dense(B)
    Gamma = O.core_gradient(W, A, B, S, Hw)
    score = np.abs(Gamma).reshape(W.shape[0], -1, 4).sum(axis=2)
    ng_row = W.shape[1] // 4
    nbo, nbi = W.shape[0] // db, W.shape[1] // db
    n_diff = 0
    for i in range(nbo):
        for j in range(nbi):
            g = info.selected[i, j]
            r, c = divmod(int(g), ng_row)
            assert i * db <= r < (i + 1) * db and j * db <= 4 * c < (j + 1) * db
            if select == O.L1_GREEDY:
                blk = score[i * db:(i + 1) * db, j * db // 4:(j + 1) * db // 4]
                assert np.isclose(score[r, c], blk.max())
            cols = np.arange(4 * c, 4 * c + 4)
            # only this group changed inside block (i, j)
            diff = (S1 != S)[i * db:(i + 1) * db, j * db:(j + 1) * db]
            diff[r - i * db, cols - j * db] = False
            assert not diff.any()
            # brute force on the full loss with everything else at its OLD value
            S0 = S.copy()
            S0[r, cols] = 0.0
            dW = (W - Ad @ S0 @ Bd) @ R
            best = (np.inf, None, None)
            for keep in itertools.combinations(range(4), 2):
                Dm = np.stack([(np.outer(Ad[:, r], Bd[cols[p]]) @ R).reshape(-1) for p in keep], axis=1)
                sol, *_ = np.linalg.lstsq(Dm, dW.reshape(-1), rcond=None)
                Lm = np.linalg.norm(dW.reshape(-1) - Dm @ sol) ** 2
                if Lm < best[0] * (1 - 1e-12):
                    best = (Lm, keep, sol)
            keep_or = tuple(np.nonzero(M1[r, cols])[0])
            if info.mask_margin[i, j] > 1e-9:
                assert keep_or == best[1]
                assert np.allclose(S1[r, cols[list(keep_or)]], best[2], rtol=1e-7, atol=1e-12)
            n_diff += keep_or != tuple(np.nonzero(M[r, cols])[0])
    assert info.groups_changed == n_diff


def test_l1_random_selection_frequencies_follow_the_scores():
    """Exponential race: P(select g) = l_g / sum l.  Chi-square over many iteration counters."""
    from scipy import stats
    rng = np.random.default_rng(12)
    db = 4
    W = rng.standard_normal((4, 4)) * 0.02
    X = rng.standard_normal((32, 4))
    H = O.gram(X)
    Hw = O.weighting(H, O.DIAG)
    oc = O.OracleConfig(db, h_mode=O.DIAG, seed=123)
    A, B, S, M = rand_state(W, H, oc, rng, scale=0.3)
    score = np.abs(O.core_gradient(W, A, B, S, Hw)).reshape(4, 1, 4).sum(axis=2).reshape(-1)
    counts = np.zeros(4)
    n = 4000
    for t in range(n):
        info = O.IterInfo()
        O.mask_step(W, A, B, S, M, Hw, oc, t, info)
        counts[int(info.selected[0, 0])] += 1
    expected = n * score / score.sum()
    chi2 = np.sum((counts - expected) ** 2 / expected)
    assert chi2 < stats.chi2.ppf(0.999, df=3)
    # a different seed gives a different stream, the same seed the same one
    i1, i2, i3 = O.IterInfo(), O.IterInfo(), O.IterInfo()
    O.mask_step(W, A, B, S, M, Hw, oc, 7, i1)
    O.mask_step(W, A, B, S, M, Hw, oc, 7, i2)
    assert np.all(i1.selected == i2.selected)


@pytest.mark.parametrize("mode", [O.L2_RANDOM, O.UNIFORM_RANDOM])
def test_ablation_selection_heuristics_follow_their_weights(mode):
    """Appendix E.1: L2-random draws a group with probability proportional to the L2 norm of its gradient,
    uniform-random with equal probability.  Chi-square over many iteration counters, as for L1-random."""
    from scipy import stats
    rng = np.random.default_rng(13)
    db = 4
    W = rng.standard_normal((4, 4)) * 0.02
    X = rng.standard_normal((32, 4))
    H = O.gram(X)
    Hw = O.weighting(H, O.DIAG)
    oc = O.OracleConfig(db, h_mode=O.DIAG, seed=321, select_mode=mode)
    A, B, S, M = rand_state(W, H, oc, rng, scale=0.3)
    Gam = O.core_gradient(W, A, B, S, Hw)
    weight = np.sqrt((Gam.reshape(4, 1, 4) ** 2).sum(axis=2)).reshape(-1) if mode == O.L2_RANDOM else np.ones(4)
    counts = np.zeros(4)
    n = 4000
    for t in range(n):
        info = O.IterInfo()
        O.mask_step(W, A, B, S, M, Hw, oc, t, info)
        counts[int(info.selected[0, 0])] += 1
    expected = n * weight / weight.sum()
    assert np.sum((counts - expected) ** 2 / expected) < stats.chi2.ppf(0.999, df=3)
    # the L1 and L2 weights differ on this input, so the two heuristics are distinguishable
    l1 = np.abs(Gam).reshape(4, 1, 4).sum(axis=2).reshape(-1)
    assert not np.allclose(l1 / l1.sum(), weight / weight.sum(), rtol=1e-2)


def test_splitmix64_reference_values():
    # first outputs of the SplitMix64 generator seeded with 0 and with 1234567
    # (published test vectors of the algorithm: state += golden gamma, then mix)
    out0 = int(O.splitmix64(np.array([0], dtype=np.uint64))[0])
    assert out0 == 0xE220A8397B1DCDAF
    s = np.uint64(1234567)
    got = []
    for _ in range(3):
        got.append(int(O.splitmix64(np.array([s], dtype=np.uint64))[0]))
        with np.errstate(over="ignore"):
            s = s + np.uint64(0x9E3779B97F4A7C15)
    assert got == [6457827717110365317, 3203168211198807973, 9817491932198370423]
    u = O.selection_uniform(3, 5, np.arange(1000, dtype=np.uint64), 1000)
    assert u.min() > 0.0 and u.max() < 1.0 and abs(u.mean() - 0.5) < 0.05


def overlapping_state(d_out=64, d_in=256, db=32, n=4, strength=0.3, seed=5):
    """A state in which the group updates of one iteration interact strongly: four calibration tokens (H has
    rank 4, so the columns of a residual row are tied together) and wrapper blocks A_i whose columns are
    nearly parallel (every group of row-block i then removes nearly the same component of E_i X^T)."""
    cfg, W, X = tiny(d_out=d_out, d_in=d_in, db=db, n=n, seed=seed)
    H = O.gram(X)
    oc = O.OracleConfig(db, h_mode=O.FULL, seed=1, phases=O.PH_MASK)
    A, B, S, M = O.init(W, H, oc)
    A = inputs.coupled_blocks(d_out // db, db, strength)
    return W, X, H, oc, (A, B, S, M)


def rebuild_discarded_update(W, X, A, B, S, info, m=4):
    """The update the oracle evaluated, rebuilt without its formulas: for every selected group (info.selected)
    and the mask chosen for it (info.new_mask), the kept values by generic least squares on the loss written
    from the activations, every other entry of S at its old value."""
    Ad, Bd = O.bd_dense(A), O.bd_dense(B)
    R = X.T
    ng_row = W.shape[1] // m
    S_new = S.copy()
    for g, bits in zip(info.selected.reshape(-1), info.new_mask.reshape(-1)):
        if g < 0:
            continue
        r, c = divmod(int(g), ng_row)
        cols = np.arange(m * c, m * c + m)
        keep = [p for p in range(m) if (int(bits) >> p) & 1]
        S0 = S.copy()
        S0[r, cols] = 0.0
        target = ((W - Ad @ S0 @ Bd) @ R).reshape(-1)
        Dm = np.stack([(np.outer(Ad[:, r], Bd[cols[p]]) @ R).reshape(-1) for p in keep], axis=1)
        sol, *_ = np.linalg.lstsq(Dm, target, rcond=None)
        S_new[r, cols] = 0.0
        S_new[r, cols[keep]] = sol
    return S_new


def test_guard_rejects_an_increase_and_keeps_the_state():
    """Full weighting: group updates that are each optimal on their own can raise the loss together.  On a
    state built to make them overlap the update MUST be discarded: the reported change is positive and equals
    the change of ||E X^T||_F^2 under the rebuilt update, each group alone would have lowered the loss
    (Lemma 2 for a single group), and the state comes back untouched."""
    W, X, H, oc, (A, B, S, M) = overlapping_state()
    Hw = O.weighting(H, O.FULL)
    L0 = loss_from_X(W, A, B, S, X)
    n_reject = 0
    for t in range(3):
        info = O.IterInfo()
        S1, M1 = O.mask_step(W, A, B, S, M, Hw, oc, t, info)
        S_try = rebuild_discarded_update(W, X, A, B, S, info)
        dL_true = loss_from_X(W, A, B, S_try, X) - L0
        assert np.isclose(info.delta_L_mask, dL_true, rtol=1e-6, atol=1e-12 * L0)
        if t < 2:                              # found by running the oracle: t = 0, 1 overshoot, t = 2 does not
            assert dL_true > 1e-3 * L0 and info.mask_accepted == 0 and info.groups_changed == 0
            assert S1 is S or np.array_equal(S1, S)
            assert M1 is M or np.array_equal(M1, M)
            n_reject += 1
            # one group of the discarded update on its own: a decrease, as Lemma 2 says
            g0 = int(info.selected[0, 0])
            one = O.IterInfo()
            one.selected = np.array([[g0]])
            one.new_mask = info.new_mask[:1, :1]
            S_one = rebuild_discarded_update(W, X, A, B, S, one)
            assert loss_from_X(W, A, B, S_one, X) <= L0 * (1 + 1e-12)
        else:
            assert info.mask_accepted == 1 and dL_true < 0 and np.allclose(S1, S_try, rtol=1e-7, atol=1e-12)
    assert n_reject == 2


def test_rejected_update_leaves_the_iteration_where_it_was():
    """Whole iterations around a rejection (sparse-core phase only): the loss after a discarded update is the
    loss before it, bit for bit, the next iteration draws other groups, and accepted updates follow
    rejected ones in the same run."""
    W, X, H, oc, state = overlapping_state()
    (A, B, S, M), infos = O.run(W, H, oc, 5, state=state)
    acc = [i.mask_accepted for i in infos]
    assert acc[:2] == [0, 0] and 1 in acc[2:]
    assert infos[0].loss["mask"] == infos[0].loss["start"] == infos[1].loss["start"]
    assert not np.array_equal(infos[0].selected, infos[1].selected)
    prev = infos[0].loss["start"]
    for i in infos:
        assert i.loss["mask"] <= prev
        assert (i.loss["mask"] < prev) == bool(i.mask_accepted and i.delta_L_mask < 0)
        prev = i.loss["mask"]
    assert np.isclose(prev, loss_from_X(W, A, B, S, X), rtol=1e-9)


def test_guard_applies_to_several_groups_per_block_with_the_diagonal_weighting():
    """With mask_groups > 1 groups of one block share columns of A or rows of B, so the joint test can fail
    with the paper's diagonal weighting as well; with one group per block it never does (Lemma 2)."""
    W, X, H, oc, (A, B, S, M) = overlapping_state(strength=1.0)
    Hw = O.weighting(H, O.DIAG)
    R = np.diag(np.sqrt(np.diag(H)))
    one = O.OracleConfig(oc.d_block, h_mode=O.DIAG, seed=1)
    many = O.OracleConfig(oc.d_block, h_mode=O.DIAG, seed=1, mask_groups=8)
    L0 = O.proxy_loss(W, A, B, S, Hw)
    seen = 0
    for t in range(6):
        i1, i8 = O.IterInfo(), O.IterInfo()
        O.mask_step(W, A, B, S, M, Hw, one, t, i1)
        assert i1.mask_accepted == 1 and i1.delta_L_mask <= 0
        S8, M8 = O.mask_step(W, A, B, S, M, Hw, many, t, i8)
        if not i8.mask_accepted:
            seen += 1
            assert i8.delta_L_mask > 0 and np.array_equal(S8, S) and np.array_equal(M8, M)
        else:
            E = W - O.bd_dense(A) @ S8 @ O.bd_dense(B)
            assert np.isclose(np.linalg.norm(E @ R) ** 2 - L0, i8.delta_L_mask, rtol=1e-6, atol=1e-12 * L0)
    assert seen >= 1


# ------------------------------------------------------------------ whole iteration
@pytest.mark.parametrize("h_mode", [O.FULL, O.DIAG])
@pytest.mark.parametrize("select", [O.L1_RANDOM, O.L1_GREEDY])
def test_theorem_1_monotone_and_below_init(h_mode, select):
    cfg, W, X = tiny(d_out=32, d_in=32, db=8, n=128)
    W, _, _ = O.normalize(W)
    H = O.gram(X)
    oc = O.OracleConfig(8, h_mode=h_mode, select_mode=select, seed=2)
    Hw = O.weighting(H, h_mode)
    L0 = O.proxy_loss(W, *O.init(W, H, oc)[:3], Hw)
    (A, B, S, M), infos = O.run(W, H, oc, 8)
    prev = L0
    for info in infos:
        assert np.isclose(info.loss["start"], prev, rtol=1e-12)
        seq = [info.loss[k] for k in ("start", "A", "B", "S", "mask")]
        for a, b in zip(seq, seq[1:]):
            assert b <= a * (1 + 1e-10)
        prev = seq[-1]
    assert prev < L0            # wrappers strictly help on this input
    assert np.all(M.reshape(32, -1, 4).sum(axis=2) == 2) and np.all(S[~M] == 0)


@pytest.mark.parametrize("n_keep", [4, 5, 6])
def test_theorem_1_with_n_of_8_groups(n_keep):
    cfg, W, X = tiny(d_out=32, d_in=32, db=8, n=128)
    H = O.gram(X)
    oc = O.OracleConfig(8, n_keep=n_keep, m_group=8, seed=3)
    L0 = O.proxy_loss(W, *O.init(W, H, oc)[:3], H)
    (A, B, S, M), infos = O.run(W, H, oc, 6)
    prev = L0
    for info in infos:
        seq = [info.loss[k] for k in ("start", "A", "B", "S", "mask")]
        assert np.isclose(seq[0], prev, rtol=1e-12)
        for a, b in zip(seq, seq[1:]):
            assert b <= a * (1 + 1e-10)
        prev = seq[-1]
    assert prev < L0
    assert np.all(M.reshape(32, -1, 8).sum(axis=2) == n_keep) and np.all(S[~M] == 0)


@pytest.mark.parametrize("h_mode", [O.FULL, O.DIAG])
def test_several_sparse_core_updates_per_iteration(h_mode):
    """mask_sweeps = K: K runs of Algorithm 3 after one continuous update.  Pinned to the single-run step,
    which has its own pins: the phase equals K mask-only iterations numbered t*K .. t*K+K-1 started from the
    state after the continuous update; K = 1 is the plain iteration; the loss (evaluated from the activations,
    not the Gram) never rises from run to run; the summed record matches the runs."""
    cfg, W, X = tiny(d_out=32, d_in=32, db=8, n=128)
    H = O.gram(X)
    Hw = O.weighting(H, h_mode)
    Xw = X if h_mode == O.FULL else np.diag(np.sqrt(np.diag(H)))
    K, t = 3, 5
    oc = O.OracleConfig(8, h_mode=h_mode, seed=6, mask_sweeps=K)
    A, B, S, M = rand_state(W, H, oc, np.random.default_rng(3), scale=0.2)
    A1, B1, S1, M1, info = O.bcd_iteration(W, A, B, S, M, Hw, oc, t)
    # the same thing by hand: continuous update only, then K single runs with their own counters
    cont = O.OracleConfig(8, h_mode=h_mode, seed=6, phases=O.PH_A | O.PH_B | O.PH_S)
    only = O.OracleConfig(8, h_mode=h_mode, seed=6, phases=O.PH_MASK)
    A2, B2, S2, M2, _ = O.bcd_iteration(W, A, B, S, M, Hw, cont, t)
    losses = [loss_from_X(W, A2, B2, S2, Xw)]
    changed = 0
    for k in range(K):
        _, _, S2, M2, sub = O.bcd_iteration(W, A2, B2, S2, M2, Hw, only, t * K + k)
        losses.append(loss_from_X(W, A2, B2, S2, Xw))
        changed += sub.groups_changed
        assert np.array_equal(sub.selected, info.sweeps[k].selected)
    assert np.array_equal(A1, A2) and np.array_equal(B1, B2) and np.array_equal(S1, S2) and np.array_equal(M1, M2)
    for a, b in zip(losses, losses[1:]):
        assert b <= a * (1 + 1e-10)
    assert losses[-1] < losses[0]
    assert len(info.sweeps) == K and info.groups_changed == changed > 0
    assert info.mask_accepted == sum(x.mask_accepted for x in info.sweeps)
    assert np.isclose(info.loss["mask"], losses[-1], rtol=1e-9)
    accepted_change = sum(x.delta_L_mask for x in info.sweeps if x.mask_accepted)
    assert np.isclose(losses[-1] - losses[0], accepted_change, rtol=1e-6, atol=1e-9 * losses[0])
    # the runs of one iteration draw different groups (different counters), and K = 1 is the plain iteration
    assert any(not np.array_equal(info.sweeps[0].selected, info.sweeps[k].selected) for k in range(1, K))
    one = O.OracleConfig(8, h_mode=h_mode, seed=6, mask_sweeps=1)
    plain = O.OracleConfig(8, h_mode=h_mode, seed=6)
    r1 = O.bcd_iteration(W, A, B, S, M, Hw, one, t)
    r0 = O.bcd_iteration(W, A, B, S, M, Hw, plain, t)
    assert all(np.array_equal(x, y) for x, y in zip(r1[:4], r0[:4]))
    assert np.all(M1.reshape(32, -1, 4).sum(axis=2) == 2) and np.all(S1[~M1] == 0)


@pytest.mark.parametrize("h_mode", [O.FULL, O.DIAG])
def test_several_groups_per_block_in_one_update(h_mode):
    """mask_groups = k: the k smallest race keys of every block are drawn and each group is solved on its own.
    Pinned to the single-group step (which has its own pins) and to the loss evaluated from the activations:
    the drawn groups are the k best keys of the block (brute force over the keys of a greedy selection, whose
    keys are the negated scores); each group's new values are what that group gets when it
    is fitted alone by least squares; the reported change of the loss is the true one; a rejected update changes
    nothing."""
    cfg, W, X = tiny(d_out=32, d_in=32, db=16, n=128)
    H = O.gram(X)
    Hw = O.weighting(H, h_mode)
    Xw = X if h_mode == O.FULL else np.diag(np.sqrt(np.diag(H)))
    k = 3
    oc = O.OracleConfig(16, h_mode=h_mode, seed=9, mask_groups=k, select_mode=O.L1_GREEDY, phases=O.PH_MASK)
    A, B, S, M = rand_state(W, H, oc, np.random.default_rng(8), scale=0.2)
    info = O.IterInfo()
    S1, M1 = O.mask_step(W, A, B, S, M, Hw, oc, 4, info)
    Gamma = O.core_gradient(W, A, B, S, Hw)
    score = np.abs(Gamma).reshape(32, 8, 4).sum(axis=2)                     # L1 norm of every group's gradient
    for i in range(2):
        for j in range(2):
            blk = score[16 * i:16 * i + 16, 4 * j:4 * j + 4]
            best = np.argsort(-blk.reshape(-1), kind="stable")[:k]
            want = sorted(int((16 * i + q // 4) * 8 + 4 * j + q % 4) for q in best)
            assert sorted(int(g) for g in info.selected_all[i, j]) == want
            assert info.selected[i, j] == info.selected_all[i, j, 0]
    L0, L1 = loss_from_X(W, A, B, S, Xw), loss_from_X(W, A, B, S1, Xw)
    if info.mask_accepted:
        assert np.isclose(L1 - L0, info.delta_L_mask, rtol=1e-7, atol=1e-9 * L0) and L1 <= L0 * (1 + 1e-12)
        # every drawn group carries the values that a least-squares fit of that group alone gives on the full loss,
        # the other groups at their old values: checked on the third pick of block (1, 0)
        g = int(info.selected_all[1, 0, 2])
        r, c = divmod(g, 8)
        cols = slice(4 * c, 4 * c + 4)
        # solve that group alone by least squares on the full loss with the other groups at their old values
        Ad, Bd_ = O.bd_dense(A), O.bd_dense(B)
        S0 = S.copy(); S0[r, cols] = 0.0
        dW = (W - Ad @ S0 @ Bd_) @ (X.T if h_mode == O.FULL else np.diag(np.sqrt(np.diag(H))))
        keep = np.nonzero(M1[r, cols])[0]
        R = X.T if h_mode == O.FULL else np.diag(np.sqrt(np.diag(H)))
        Dm = np.stack([(np.outer(Ad[:, r], Bd_[4 * c + p_]) @ R).reshape(-1) for p_ in keep], axis=1)
        sol, *_ = np.linalg.lstsq(Dm, dW.reshape(-1), rcond=None)
        assert np.allclose(S1[r, cols][keep], sol, rtol=1e-6, atol=1e-10)
    else:
        assert np.array_equal(S1, S) and np.array_equal(M1, M)
    assert np.all(M1.reshape(32, -1, 4).sum(axis=2) == 2) and np.all(S1[~M1] == 0.0)
    # k = 1 is the plain step
    a = O.mask_step(W, A, B, S, M, Hw, O.OracleConfig(16, h_mode=h_mode, seed=9, mask_groups=1, phases=O.PH_MASK), 4)
    b = O.mask_step(W, A, B, S, M, Hw, O.OracleConfig(16, h_mode=h_mode, seed=9, phases=O.PH_MASK), 4)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_theorem_1_with_several_groups_per_block():
    cfg, W, X = tiny(d_out=32, d_in=32, db=8, n=128)
    H = O.gram(X)
    for h_mode in (O.FULL, O.DIAG):
        Hw = O.weighting(H, h_mode)
        oc = O.OracleConfig(8, h_mode=h_mode, seed=5, mask_groups=4)
        L0 = O.proxy_loss(W, *O.init(W, H, oc)[:3], Hw)
        (A, B, S, M), infos = O.run(W, H, oc, 6)
        prev = L0
        for info in infos:
            seq = [info.loss[k_] for k_ in ("start", "A", "B", "S", "mask")]
            assert np.isclose(seq[0], prev, rtol=1e-12)
            for a, b in zip(seq, seq[1:]):
                assert b <= a * (1 + 1e-10)
            prev = seq[-1]
        assert prev < L0 and sum(i.groups_changed for i in infos) > 0
        assert np.all(M.reshape(32, -1, 4).sum(axis=2) == 2) and np.all(S[~M] == 0)


# ------------------------------------------------------------------ the paper's gradient steps (Algorithm 2)
def _grad_fd(f, X, eps=1e-6):
    g = np.zeros_like(X)
    it = np.nditer(X, flags=["multi_index"])
    for _ in it:
        ix = it.multi_index
        Xp, Xm = X.copy(), X.copy()
        Xp[ix] += eps
        Xm[ix] -= eps
        g[ix] = (f(Xp) - f(Xm)) / (2 * eps)
    return g


def test_gradient_steps_follow_finite_differences_and_the_descent_lemma():
    """A and B updates of Algorithm 2 with the steps of Eq. lrA / lrB: the move is -eta * gradient with the
    gradient checked by central differences, beta bounds the change of the gradient between two points, and the
    loss drops by at least ||grad||^2 / (2 beta) (descent lemma for a beta-smooth function)."""
    cfg, W, X = tiny(d_out=8, d_in=12, db=4, n=60)
    H = O.gram(X)
    Hw = O.weighting(H, O.DIAG)
    oc = O.OracleConfig(4, h_mode=O.DIAG, ab_step=O.AB_GD)
    rng = np.random.default_rng(20)
    A, B, S, M = rand_state(W, H, oc, rng, scale=0.3)
    L0 = O.proxy_loss(W, A, B, S, Hw)
    # ---- A
    gA = _grad_fd(lambda Z: O.proxy_loss(W, Z, B, S, Hw), A)
    A1, tauA = O.a_step_gd(W, A, B, S, Hw, oc)
    assert np.allclose(A1 - A, -0.5 * tauA * gA, rtol=1e-5, atol=1e-9 * np.abs(gA).max())
    betaA = 2.0 / tauA
    A2 = A + 0.2 * rng.standard_normal(A.shape)
    gA2 = _grad_fd(lambda Z: O.proxy_loss(W, Z, B, S, Hw), A2)
    assert np.linalg.norm(gA - gA2) <= betaA * np.linalg.norm(A - A2) * (1 + 1e-6)
    LA = O.proxy_loss(W, A1, B, S, Hw)
    assert LA <= L0 - np.sum(gA * gA) / (2 * betaA) * (1 - 1e-6)
    # ---- B, from the new A
    gB = _grad_fd(lambda Z: O.proxy_loss(W, A1, Z, S, Hw), B)
    B1, tauB = O.b_step_gd(W, A1, B, S, Hw, oc)
    assert np.allclose(B1 - B, -0.5 * tauB * gB, rtol=1e-5, atol=1e-9 * np.abs(gB).max())
    betaB = 2.0 / tauB
    B2 = B + 0.2 * rng.standard_normal(B.shape)
    gB2 = _grad_fd(lambda Z: O.proxy_loss(W, A1, Z, S, Hw), B2)
    assert np.linalg.norm(gB - gB2) <= betaB * np.linalg.norm(B - B2) * (1 + 1e-6)
    assert O.proxy_loss(W, A1, B1, S, Hw) <= LA - np.sum(gB * gB) / (2 * betaB) * (1 - 1e-6)


def test_theorem_1_for_the_papers_literal_continuous_update():
    """Algorithm 1 with Algorithm 2 as printed: gradient steps for A, B and W' with the 1/beta steps, diagonal
    weighting.  Lemma 1 / Theorem 1: the loss never increases and never exceeds the initialisation's."""
    cfg, W, X = tiny(d_out=32, d_in=32, db=8, n=128)
    H = O.gram(X)
    oc = O.OracleConfig(8, h_mode=O.DIAG, ab_step=O.AB_GD, s_step=O.S_BETA, seed=4)
    Hw = O.weighting(H, O.DIAG)
    L0 = O.proxy_loss(W, *O.init(W, H, oc)[:3], Hw)
    (A, B, S, M), infos = O.run(W, H, oc, 12)
    prev = L0
    for info in infos:
        seq = [info.loss[k] for k in ("start", "A", "B", "S", "mask")]
        assert np.isclose(seq[0], prev, rtol=1e-12)
        for a, b in zip(seq, seq[1:]):
            assert b <= a * (1 + 1e-12)
        assert info.tau_A > 0 and info.tau_B > 0
        prev = seq[-1]
    assert prev < L0
    with pytest.raises(ValueError):
        O.bcd_iteration(W, A, B, S, M, H, O.OracleConfig(8, h_mode=O.FULL, ab_step=O.AB_GD), 0)


def test_joint_adam_step_properties():
    """The joint Adam step (Section 3.3.1; Kingma & Ba, Algorithm 1), pinned by what the algorithm's definition
    fixes: (1) with zero moments the bias-corrected first step moves every entry by lr * sign(gradient);
    (2) the three gradients are taken at the same point (A's move follows the finite-difference gradient at
    the OLD B and W'); (3) masked-out entries of W' never move; (4) a constant gradient keeps the step at lr;
    (5) the second step follows the recurrences written out by hand for one entry."""
    cfg, W, X = tiny(d_out=8, d_in=12, db=4, n=60)
    H = O.gram(X)
    Hw = O.weighting(H, O.FULL)
    oc = O.OracleConfig(4, ab_step=O.AB_ADAM, adam_lr=1e-3, adam_eps=1e-30)
    rng = np.random.default_rng(21)
    A, B, S, M = rand_state(W, H, oc, rng, scale=0.3)
    st = O.adam_state(A, B, S)
    gA_fd = _grad_fd(lambda Z: O.proxy_loss(W, Z, B, S, Hw), A)
    gB_fd = _grad_fd(lambda Z: O.proxy_loss(W, A, Z, S, Hw), B)
    gS_fd = _grad_fd(lambda Z: O.proxy_loss(W, A, B, Z * M, Hw), S)
    gA, gB, gS = O.joint_gradients(W, A, B, S, M, Hw, oc)
    for g, fd in ((gA, gA_fd), (gB, gB_fd), (gS, gS_fd)):
        assert np.allclose(g, fd, rtol=1e-5, atol=1e-8 * np.abs(fd).max())
    A1, B1, S1 = O.adam_joint_step(W, A, B, S, M, Hw, oc, st, 1)
    assert np.allclose(A1 - A, -1e-3 * np.sign(gA_fd), rtol=1e-9)
    assert np.allclose(B1 - B, -1e-3 * np.sign(gB_fd), rtol=1e-9)
    assert np.allclose((S1 - S)[M], -1e-3 * np.sign(gS_fd[M]), rtol=1e-9)
    assert np.all((S1 - S)[~M] == 0.0) and np.all(S1[~M] == 0.0)
    # second step: recurrences by hand for one entry of A
    g1 = gA[0, 1, 2]
    g2 = O.joint_gradients(W, A1, B1, S1, M, Hw, oc)[0][0, 1, 2]
    A2, _, _ = O.adam_joint_step(W, A1, B1, S1, M, Hw, oc, st, 2)
    m2 = 0.9 * (0.1 * g1) + 0.1 * g2
    v2 = 0.999 * (0.001 * g1 * g1) + 0.001 * g2 * g2
    step = 1e-3 * (m2 / (1 - 0.9 ** 2)) / np.sqrt(v2 / (1 - 0.999 ** 2))
    assert np.isclose(A2[0, 1, 2], A1[0, 1, 2] - step, rtol=1e-12, atol=0.0)
    # a constant gradient: the step stays lr (quadratic with A only, far from its minimum along a fixed sign)
    oc_eps = O.OracleConfig(4, ab_step=O.AB_ADAM, adam_lr=1e-6, adam_eps=1e-30)
    st2 = O.adam_state(A, B, S)
    Ak, Bk, Sk = A, B, S
    for t in range(1, 4):
        An, Bn, Sn = O.adam_joint_step(W, Ak, Bk, Sk, M, Hw, oc_eps, st2, t)
        assert np.allclose(np.abs(An - Ak), 1e-6, rtol=1e-3)     # gradients barely change over 1e-6 moves
        Ak, Bk, Sk = An, Bn, Sn


def test_joint_adam_run_lowers_the_loss_and_keeps_the_pattern():
    cfg, W, X = tiny(d_out=32, d_in=32, db=8, n=128)
    H = O.gram(X)
    oc = O.OracleConfig(8, h_mode=O.DIAG, ab_step=O.AB_ADAM, adam_lr=1e-3, seed=5)
    Hw = O.weighting(H, O.DIAG)
    L0 = O.proxy_loss(W, *O.init(W, H, oc)[:3], Hw)
    (A, B, S, M), infos = O.run(W, H, oc, 40)
    assert infos[-1].loss["mask"] < 0.9 * L0
    for info in infos:      # the sparse-core update itself never raises the loss (Lemma 2), whatever Adam did before
        assert info.loss["mask"] <= info.loss["S"] * (1 + 1e-12)
    assert np.all(M.reshape(32, -1, 4).sum(axis=2) == 2) and np.all(S[~M] == 0)


def test_resume_is_bitwise():
    cfg, W, X = tiny(d_out=16, d_in=16, db=8, n=64)
    H = O.gram(X)
    oc = O.OracleConfig(8, seed=9)
    full, _ = O.run(W, H, oc, 6, want_loss=False)
    half, _ = O.run(W, H, oc, 3, want_loss=False)
    rest, _ = O.run(W, H, oc, 3, t_first=3, state=half, want_loss=False)
    for a, b in zip(full, rest):
        assert np.array_equal(a, b)


def test_diagonal_wrappers_cannot_beat_the_init():
    """Appendix A: diag(a) (W'.M) diag(b) = W''.M, so diagonal-only wrappers add nothing
    and the loss cannot drop below the optimum for A = B = I (DIAG mode)."""
    cfg, W, X = tiny()
    H = O.gram(X)
    oc = O.OracleConfig(cfg.d_block, h_mode=O.DIAG)
    Hw = O.weighting(H, O.DIAG)
    A, B, S, M = O.init(W, H, oc)
    L0 = O.proxy_loss(W, A, B, S, Hw)
    rng = np.random.default_rng(14)
    for _ in range(20):
        a = 1 + 0.3 * rng.standard_normal(W.shape[0])
        b = 1 + 0.3 * rng.standard_normal(W.shape[1])
        Ad = np.stack([np.diag(a[i * 8:(i + 1) * 8]) for i in range(A.shape[0])])
        Bd = np.stack([np.diag(b[j * 8:(j + 1) * 8]) for j in range(B.shape[0])])
        Sr = (S + 0.01 * rng.standard_normal(S.shape)) * M
        lhs = O.bd_dense(Ad) @ Sr @ O.bd_dense(Bd)
        assert np.allclose(lhs, (a[:, None] * Sr * b[None, :]) * M)
        assert O.proxy_loss(W, Ad, Bd, Sr, Hw) >= L0 * (1 - 1e-12)


# ------------------------------------------------------------------ apply, storage
def test_apply_equals_dense_product_and_denormalisation():
    cfg, W, X = tiny()
    Wb, r1, r2 = O.normalize(W)
    H = O.gram(X)
    oc = O.OracleConfig(cfg.d_block)
    A, B, S, M = rand_state(Wb, H, oc, np.random.default_rng(15))
    x = X[:7]
    What = O.bd_dense(A) @ S @ O.bd_dense(B)
    assert np.allclose(O.apply(A, B, S, x), x @ What.T, rtol=1e-10)
    full = np.diag(r2) @ What @ np.diag(r1)
    assert np.allclose(O.apply(A, B, S, x, r1, r2), x @ full.T, rtol=1e-10)
    # with the init state and no pruning error the de-normalised product returns W x
    A0, B0, _, _ = O.init(Wb, H, oc)
    assert np.allclose(O.apply(A0, B0, Wb, x, r1, r2), x @ W.T, rtol=1e-9)


def test_overhead_percentages_printed_in_the_paper():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "overhead.txt")) if l.strip() and not l.startswith("#")]
    for name, shapes, want in rows:
        tot_w = tot_o = 0
        for sh in shapes.split(";"):
            cnt, dims = sh.split("*")
            d_out, d_in = (int(v) for v in dims.split("x"))
            tot_w += int(cnt) * d_out * d_in
            tot_o += int(cnt) * O.overhead_fraction(d_out, d_in, 128) * d_out * d_in
        assert abs(100 * tot_o / tot_w - float(want)) < 0.006, name
