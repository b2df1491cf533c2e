"""Construction of the per-block WUSH transforms (Algorithm 1, Eq. 5-6).

Test infrastructure (see the package docstring).  Notation follows the paper:
M_W, M_X are the d x d second moments of one block of weights / calibration
activations, W', X' their lower Cholesky factors, U S V^T the SVD of W'^T X',
H the normalised Hadamard matrix, and

    T_wush = H S^-1/2 U^T W'^T      (multiplies ACTIVATIONS online, Eq. 7)
    T_xvsh = H S^-1/2 V^T X'^T      (multiplies WEIGHTS offline, Algorithm 2)
    T_xvsh = T_wush^-T              (Eq. 6)
"""
import numpy as np

from . import formats as F


def hadamard(d):
    """Normalised Sylvester-Hadamard matrix: H[i,j] = (-1)^popcount(i & j) / sqrt(d)."""
    if d < 1 or d & (d - 1):
        raise ValueError("d must be a power of two")
    idx = np.arange(d)
    anded = idx[:, None] & idx[None, :]
    pop = np.zeros((d, d), dtype=np.int64)
    for b in range(max(1, d.bit_length())):
        pop += (anded >> b) & 1
    return np.where(pop % 2 == 0, 1.0, -1.0) / np.sqrt(d)


def damped(M, lam):
    """M + lam * d^-1 tr(M) I  (the argument of both Cholesky steps in Algorithm 1)."""
    d = M.shape[0]
    return M + lam * np.trace(M) / d * np.eye(d)


def wush_block(M_W, M_X, lam=0.01, return_parts=False):
    """Algorithm 1 for one block.  Returns T_wush (fp64, d x d).

    The SVD is unique only up to the sign of each singular pair (and order of equal
    singular values); Lemma A.1 shows the product U^T W'^T is the factor-independent
    quantity, so the convention is fixed there: singular values descending, and each
    row of U^T W'^T has its largest-magnitude entry positive.
    """
    M_W = np.asarray(M_W, dtype=np.float64)
    M_X = np.asarray(M_X, dtype=np.float64)
    d = M_W.shape[0]
    H = hadamard(d)
    Wp = np.linalg.cholesky(damped(M_W, lam))          # W' W'^T = damped M_W, W' lower
    Xp = np.linalg.cholesky(damped(M_X, lam))          # X' X'^T = damped M_X
    U, S, Vt = np.linalg.svd(Wp.T @ Xp)                # W'^T X' = U S V^T, S descending
    UtWt = U.T @ Wp.T
    pick = np.argmax(np.abs(UtWt), axis=1)
    sgn = np.sign(UtWt[np.arange(d), pick])
    sgn[sgn == 0] = 1.0
    UtWt = UtWt * sgn[:, None]
    T = H @ (UtWt / np.sqrt(S)[:, None])               # H S^-1/2 U^T W'^T
    if return_parts:
        U = U * sgn[None, :]
        Vt = Vt * sgn[:, None]
        return T, dict(H=H, Wp=Wp, Xp=Xp, U=U, S=S, Vt=Vt)
    return T


def xvsh_from_wush(T_wush):
    """T_xvsh = T_wush^-T (Eq. 6): the weight-side partner of an activation transform."""
    return np.linalg.inv(np.asarray(T_wush, dtype=np.float64)).T


def build_transforms(mom_W, mom_X, lam=0.01):
    """Algorithm 2, RTN case, lines 'WUSH' and 'T_xvsh <- T_wush^-T', for all blocks.

    mom_W, mom_X: [C, d, d] normalised second moments.  Returns
      T_hat_bits  uint16 [C, d, d]  bf16 storage of T_wush ("16-bit transforms"),
      T_hat       fp64   [C, d, d]  the values those bits decode to,
      T_xvsh      fp64   [C, d, d]  inverse-transpose of the ROUNDED T_hat, so that
                                    (x T_hat^T)(w T_xvsh^T)^T = x w^T holds exactly.
    """
    C = mom_W.shape[0]
    T = np.stack([wush_block(mom_W[c], mom_X[c], lam) for c in range(C)])
    bits = F.f64_to_bf16_bits(T)
    That = F.bf16_bits_to_f64(bits)
    Tx = np.ascontiguousarray(np.stack([xvsh_from_wush(That[c]) for c in range(C)]))
    return bits, That, Tx


# Comparison transforms of Table 1 (used only by the qualitative ordering test).
def variant_transform(kind, M_W, M_X, lam=0.01, rng=None):
    d = M_W.shape[0]
    if kind == "I":
        return np.eye(d)
    if kind == "H":
        return hadamard(d)
    if kind == "R":
        q, r = np.linalg.qr(rng.standard_normal((d, d)))
        return q * np.sign(np.diag(r))[None, :]
    if kind == "WUS":                                   # WUSH without the Hadamard factor
        return hadamard(d).T @ wush_block(M_W, M_X, lam)
    if kind == "WUSH":
        return wush_block(M_W, M_X, lam)
    raise ValueError(kind)
