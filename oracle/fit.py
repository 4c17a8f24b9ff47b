"""CPU oracle (test infrastructure): basis fit and bit allocation, fp64 numpy.

Transform (method Sec. 3.1, Eq. 3-4).  The paper factorises the key projection through the
SVD of the whitened weight M = G^{1/2} W = U S V^T.  The second moment of the keys the model
produces is E[k^T k] = W^T G W = M^T M = V S^2 V^T, so V is the eigenbasis of the *uncentred*
second moment of the produced keys and the eigenvalues are the squared singular values.  At
full rank the paper's latent is c = (k V) S^{-1/2} with E[c^T c] = S (Eq. 4), and the key is
recovered as c S^{1/2} V^T.  This module fits exactly that from cache vectors:

    C = X^T X / N (uncentred), mu = mean(X);  C = U diag(lam) U^T, lam descending
    m = mu U                      (measured coordinate means, removed before quantisation)
    var_j = max(lam_j - m_j^2, 0) (centred marginal variance of rotated coordinate j)
    gains: ROTATE gamma = 1; SQRT gamma_j = lam_j^{-1/4} (the paper's square-root split: the
           stored coordinate has second moment lam_j^{1/2}); WHITEN gamma_j = var_j^{-1/2}
           (the footnote's pure-whitening alternative)
    W_enc = U diag(gamma), W_dec = diag(1/gamma) U^T, m' = m * gamma

Allocation (Sec. 3.2, Eq. 5, appendix "Reverse water-filling derivation"): minimise
sum_j v_j 4^{-b_j} at a fixed total rate, widths clamped to [0, b_max].  The closed form is
Eq. 5; the integer realisation used by the codec is the exact integer minimiser found by
greedy marginal return (each added bit divides a channel's distortion by 4).

The eigendecomposition uses numpy.linalg.eigh as a library step.
"""
import numpy as np

GAIN_ROTATE, GAIN_SQRT, GAIN_WHITEN = 0, 1, 2
EPS_FLOOR = 1e-12


def second_moment(X):
    """Uncentred second moment C = X^T X / N and mean, fp64 (Sec. 3 preamble: G = E[h^T h])."""
    X = np.asarray(X, dtype=np.float64)
    n = X.shape[0]
    return X.T @ X / n, X.sum(axis=0) / n


def eig_descending(C):
    """Symmetric eigendecomposition, eigenvalues descending, each eigenvector's largest-magnitude
    component made positive (ties: lowest index)."""
    lam, U = np.linalg.eigh(np.asarray(C, dtype=np.float64))
    order = np.argsort(-lam, kind="stable")
    lam = lam[order]
    U = U[:, order]
    for j in range(U.shape[1]):
        k = int(np.argmax(np.abs(U[:, j])))
        if U[k, j] < 0:
            U[:, j] = -U[:, j]
    return lam, U


def fit_from_moments(C, mu, gain_mode=GAIN_SQRT):
    lam, U = eig_descending(C)
    lam = np.maximum(lam, 0.0)
    m = mu @ U
    var = np.maximum(lam - m * m, 0.0)
    floor = EPS_FLOOR * lam[0]
    if gain_mode == GAIN_ROTATE:
        gamma = np.ones_like(lam)
    elif gain_mode == GAIN_SQRT:
        gamma = np.maximum(lam, floor) ** -0.25
    elif gain_mode == GAIN_WHITEN:
        gamma = np.maximum(var, floor) ** -0.5
    else:
        raise ValueError("gain_mode")
    W_enc = U * gamma[None, :]
    W_dec = (U / gamma[None, :]).T
    m_rot = m * gamma
    v_alloc = var if gain_mode == GAIN_WHITEN else var * gamma * gamma
    return dict(U=U, lam=lam, mu=mu, m=m, var=var, gamma=gamma, W_enc=W_enc, W_dec=W_dec, m_rot=m_rot,
                v_alloc=v_alloc)


def fit_basis(X, gain_mode=GAIN_SQRT):
    C, mu = second_moment(X)
    out = fit_from_moments(C, mu, gain_mode)
    out["C"] = C
    return out


# ------------------------------------------------------------------ allocation

def total_bits(d, ratio):
    """Payload bits per token per unit-side for a nominal ratio against 16-bit elements."""
    return int(np.floor(16.0 * d / ratio + 1e-9))


def waterfill_closed_form(v, b_mean, b_max):
    """Eq. 5 with the clamp to [0, b_max]: b_j = b_mean + 0.5 log2(v_j / GM(v)) on the unclamped set,
    re-solved until the set is stable so that the mean rate is met.  Real-valued."""
    v = np.asarray(v, dtype=np.float64)
    r = v.size
    b = np.zeros(r)
    free = v > 0
    fixed_hi = np.zeros(r, dtype=bool)
    budget = b_mean * r
    for _ in range(4 * r + 4):
        idx = np.where(free & ~fixed_hi)[0]
        if idx.size == 0:
            break
        rem = budget - b_max * fixed_hi.sum()
        logv = np.log2(v[idx])
        bb = rem / idx.size + 0.5 * (logv - logv.mean())
        if (bb < 0).any():
            free[idx[np.argmin(bb)]] = False
            continue
        if (bb > b_max).any():
            fixed_hi[idx[np.argmax(bb)]] = True
            continue
        b[:] = 0
        b[idx] = bb
        b[fixed_hi] = b_max
        return b
    b[:] = 0
    b[fixed_hi] = b_max
    return b


def alloc_bits(v, btot, b_max=8, width_group=1):
    """Integer widths: exact minimiser of sum_j v_j 4^{-b_j} subject to sum b_j <= btot, 0 <= b_j <= b_max,
    channels in groups of `width_group` sharing one width taken from the group's mean variance (Sec. 3.2).
    Greedy: btot // width_group times, give one bit to the group with the largest current v_G 4^{-b_G} among
    those below b_max (ties: lowest index).  Comparison values are the fp32 inputs scaled by exact powers of
    four, held in fp64."""
    v32 = np.asarray(v, dtype=np.float32)
    d = v32.size
    ng = d // width_group
    if width_group == 1:
        vg = v32.astype(np.float64)
    else:
        # group mean, summed in fp32 in index order then divided in fp32 (matches a plain loop)
        vg = np.empty(ng, dtype=np.float64)
        for g in range(ng):
            acc = np.float32(0)
            for j in range(g * width_group, (g + 1) * width_group):
                acc = np.float32(acc + v32[j])
            vg[g] = np.float64(np.float32(acc / np.float32(width_group)))
    b = np.zeros(ng, dtype=np.int64)
    steps = min(btot // width_group, ng * b_max)
    for _ in range(steps):
        best, best_val = -1, -1.0
        for g in range(ng):
            if b[g] >= b_max:
                continue
            val = vg[g] * 4.0 ** (-int(b[g]))
            if val > best_val:
                best, best_val = g, val
        b[best] += 1
    return np.repeat(b, width_group).astype(np.uint8)


def alloc_bits_pooled(v_units, btot_per_unit, b_max=8, width_group=1):
    """The same allocation with the budget pooled over several units (the KV heads of a layer: the paper's latent
    spans all of them, Sec. 3.2 and the appendix's bit-profile figure).  v_units [n, d]; the n * d channels compete
    for n * btot_per_unit bits under the rule of alloc_bits (index order: unit, then channel).  Returns [n, d]."""
    v_units = np.asarray(v_units, dtype=np.float32)
    n, d = v_units.shape
    return alloc_bits(v_units.reshape(-1), n * btot_per_unit, b_max, width_group).reshape(n, d)


def split_ratio(ratio, kappa):
    """Key/value budget split (Sec. 3.1, last paragraph; appendix on hyperparameters): keys get the fraction kappa of
    the bits that `ratio` gives keys and values together.  Returns (ratio_k, ratio_v)."""
    return ratio / (2.0 * kappa), ratio / (2.0 * (1.0 - kappa))


# ------------------------------------------------------------------ rate accounting

def effective_bits_per_element(widths, scale_group):
    """Stored bits per original element: payload plus one fp16 scale and one fp16 zero-point per token per
    active scale group (appendix "Effective compression ratio")."""
    widths = np.asarray(widths)
    d = widths.size
    n_act = sum(1 for g in range(d // scale_group) if widths[g * scale_group:(g + 1) * scale_group].any())
    return (widths.sum() + 32.0 * n_act) / d


def effective_ratio(widths, scale_group):
    return 16.0 / effective_bits_per_element(widths, scale_group)


def max_context_tokens(budget_gib, ratio, weights_gb=16.06, dense_bytes_per_token=131072):
    """Longest single-sequence context that fits: (budget - resident weights) / (dense bytes per token / ratio)
    (appendix table "Max single-sequence context vs GPU memory budget"; budget and weights in units of 2^30 B)."""
    return (budget_gib - weights_gb) * 2.0 ** 30 / (dense_bytes_per_token / ratio)
