"""Pins for the oracle's transform construction (Algorithm 1) - CPU only.

The paper prints no worked numbers for Algorithm 1, so the construction is pinned
by the identities it proves: Eq. 6, the equalisation identity of the appendix, the
moment-matching property that is independent of the SVD's sign/order freedom,
Lemma A.1 (independence of the square-root factor), a diagonal closed form, and
the Monte-Carlo optimum of Theorem 4.1 under the paper's FP noise model.
"""
import numpy as np
import pytest
import scipy.linalg

from oracle import wush_transform as WT


def _moments(d, seed, outlier=True, B=512, N=1024):
    rng = np.random.default_rng(seed)
    s = np.exp(0.5 * rng.standard_normal(d))
    if outlier:
        s[3] *= 50
    mix = np.eye(d) + 0.3 * rng.standard_normal((d, d)) / np.sqrt(d)      # correlated channels
    X = (rng.standard_normal((B, d)) * s) @ mix
    W = 0.02 * rng.standard_normal((N, d)) @ np.linalg.inv(mix).T * np.exp(0.3 * rng.standard_normal((N, 1)))
    return W.T @ W / N, X.T @ X / B, W, X


@pytest.mark.parametrize("d", [1, 2, 16, 32, 64])
def test_hadamard(d):
    H = WT.hadamard(d)
    assert np.allclose(H @ H.T, np.eye(d), atol=1e-14)
    assert np.array_equal(H, H.T)
    assert np.allclose(np.abs(H), d ** -0.5)
    assert np.array_equal(np.sign(H), scipy.linalg.hadamard(d))           # library Sylvester construction
    assert np.allclose((H * np.sqrt(d)) @ (H * np.sqrt(d)).T, d * np.eye(d))


@pytest.mark.parametrize("d", [16, 32])
@pytest.mark.parametrize("lam", [0.0, 0.01])
def test_wush_identities(d, lam):
    MW, MX, _, _ = _moments(d, 10 + d)
    T, p = WT.wush_block(MW, MX, lam, return_parts=True)
    Tx = WT.xvsh_from_wush(T)
    H, S = p["H"], p["S"]
    MWd, MXd = WT.damped(MW, lam), WT.damped(MX, lam)
    I = np.eye(d)
    # Eq. 6: T_xvsh T_wush^T = I, and T_xvsh equals its own closed form H S^-1/2 V^T X'^T
    assert np.allclose(Tx @ T.T, I, atol=1e-9)
    Tx_closed = H @ np.diag(S ** -0.5) @ p["Vt"] @ p["Xp"].T
    assert np.allclose(Tx, Tx_closed, rtol=1e-7, atol=1e-9 * np.abs(Tx).max())
    # equalisation: T_wush M_X T_wush^T = H S H^T = T_xvsh M_W T_xvsh^T, constant diagonal tr(S)/d
    HSH = H @ np.diag(S) @ H.T
    A = T @ MXd @ T.T
    B = Tx @ MWd @ Tx.T
    assert np.allclose(A, HSH, rtol=1e-8, atol=1e-10 * S.max())
    assert np.allclose(B, HSH, rtol=1e-8, atol=1e-10 * S.max())
    assert np.allclose(np.diag(A), S.sum() / d, rtol=1e-8)
    # moment matching (independent of SVD sign / order): G = T^T T satisfies G M_X G = M_W
    G = T.T @ T
    assert np.allclose(G @ MXd @ G, MWd, rtol=1e-7, atol=1e-9 * np.abs(MWd).max())
    # singular values sorted, convention: largest entry of each row of U^T W'^T positive
    assert np.all(np.diff(S) <= 0)
    R = np.sqrt(S)[:, None] * (H.T @ T)
    assert np.all(R[np.arange(d), np.abs(R).argmax(axis=1)] > 0)


def test_wush_diagonal_closed_form():
    rng = np.random.default_rng(7)
    d = 16
    a = np.exp(rng.standard_normal(d))
    b = np.exp(rng.standard_normal(d))
    T = WT.wush_block(np.diag(a), np.diag(b), lam=0.0)
    # W' = diag(sqrt a), X' = diag(sqrt b): singular values sqrt(a_j b_j); T = H P^T diag((a/b)^1/4)
    order = np.argsort(-np.sqrt(a * b))
    P = np.eye(d)[:, order]
    closed = WT.hadamard(d) @ P.T @ np.diag((a / b) ** 0.25)
    assert np.allclose(T, closed, rtol=1e-10, atol=1e-12)


def test_wush_independent_of_square_root_factor():
    """Lemma A.1: replacing the Cholesky factors by symmetric square roots leaves T unchanged."""
    d = 16
    MW, MX, _, _ = _moments(d, 21)
    T_chol = WT.wush_block(MW, MX, 0.01)

    def sym_sqrt(M):
        w, V = np.linalg.eigh(M)
        return V @ np.diag(np.sqrt(w)) @ V.T

    Wp, Xp = sym_sqrt(WT.damped(MW, 0.01)), sym_sqrt(WT.damped(MX, 0.01))
    U, S, Vt = np.linalg.svd(Wp.T @ Xp)
    UtWt = U.T @ Wp.T
    sgn = np.sign(UtWt[np.arange(d), np.abs(UtWt).argmax(axis=1)])
    T_sym = WT.hadamard(d) @ (UtWt * sgn[:, None] / np.sqrt(S)[:, None])
    assert np.allclose(T_chol, T_sym, rtol=1e-8, atol=1e-10 * np.abs(T_chol).max())


def test_theorem_optimum_under_fp_noise_model():
    """Theorem 4.1 / FP model: E||T^-1 eps(T y)||^2 with eps_j = eta_j (T y)_j.

    For y = X' z (so that T y has second moment H S H^T), the paper's optimum gives
    E[eta^2] (tr S)^2 / d, while any orthogonal T applied to the symmetrised problem
    gives E[eta^2] tr(S^2).  Checked by Monte Carlo on the output-space loss
    || W'^T T^-1 eps ||^2 with the construction from Algorithm 1.
    """
    d = 16
    rng = np.random.default_rng(8)
    MW, MX, _, _ = _moments(d, 33, outlier=True)
    T, p = WT.wush_block(MW, MX, 0.0, return_parts=True)
    Wp, Xp, S = p["Wp"], p["Xp"], p["S"]
    n = 200000
    z = rng.standard_normal((n, d))
    y = z @ Xp.T                                       # rows: activation samples with moment M_X
    eta = rng.uniform(-1, 1, (n, d)) * 0.05
    eta2 = (0.05 ** 2) / 3

    def loss(Tm):
        ty = y @ Tm.T
        err = (eta * ty) @ np.linalg.inv(Tm).T         # T^-1 eps, back in activation space
        out = err @ Wp                                 # W'^T-weighted output error
        return np.mean(np.sum(out ** 2, axis=1))

    l_wush = loss(T)
    l_id = loss(np.eye(d))
    l_had = loss(WT.hadamard(d))
    assert abs(l_wush - eta2 * S.sum() ** 2 / d) / l_wush < 0.03
    assert l_wush < l_had and l_wush < l_id
    # no other transform of the same family (random rotations in place of H) does better
    for k in range(5):
        Rr = WT.variant_transform("R", MW, MX, rng=rng)
        assert loss(Rr.T @ WT.hadamard(d).T @ T) >= l_wush * 0.98


def test_build_transforms_rounding_and_pairing():
    d, C = 32, 3
    moms = [_moments(d, 40 + c) for c in range(C)]
    mW = np.stack([m[0] for m in moms]); mX = np.stack([m[1] for m in moms])
    bits, That, Tx = WT.build_transforms(mW, mX, 0.01)
    assert bits.dtype == np.uint16 and bits.shape == (C, d, d)
    T = np.stack([WT.wush_block(mW[c], mX[c], 0.01) for c in range(C)])
    assert np.all(np.abs(That - T) <= np.abs(T) * 2.0 ** -8 + 1e-300)     # bf16: 8 significant bits
    for c in range(C):
        assert np.allclose(Tx[c] @ That[c].T, np.eye(d), atol=1e-9)       # pairing uses the ROUNDED transform
