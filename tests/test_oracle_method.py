"""Pins for the oracle's basis fit, bit allocation, rate accounting and attention (CPU only)."""
import itertools
import os

import math

import numpy as np
import pytest

import spectra_inputs as si
from oracle import codec, fit

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _tiny_side(side, n=1024):
    wl = si.WORKLOADS["tiny"]
    return si.draw_unit(wl, 0, 0, side, 0, n_tokens=n).astype(np.float64)


# ----------------------------------------------------------------------------- basis

@pytest.mark.parametrize("mode", [fit.GAIN_ROTATE, fit.GAIN_SQRT, fit.GAIN_WHITEN])
def test_basis_is_orthonormal_and_diagonalises(mode):
    X = _tiny_side(si.SIDE_K)
    f = fit.fit_basis(X, mode)
    U, lam, C = f["U"], f["lam"], f["C"]
    d = U.shape[0]
    assert np.abs(U.T @ U - np.eye(d)).max() <= 1e-10
    off = U.T @ C @ U - np.diag(lam)
    assert np.abs(off).max() <= 1e-12 * np.abs(C).max() * d
    assert (np.diff(lam) <= 1e-15 * lam[0]).all()
    assert np.abs(f["W_enc"] @ f["W_dec"] - np.eye(d)).max() <= 1e-10
    # each eigenvector's largest component is positive (sign convention)
    assert (U[np.argmax(np.abs(U), axis=0), np.arange(d)] > 0).all()


def test_basis_recovers_a_constructed_spectrum():
    """X = sqrt(N) diag(sqrt(lam)) Q^T with N = d has X^T X / N = Q diag(lam) Q^T exactly."""
    rng = np.random.default_rng(2)
    d = 32
    q, _ = np.linalg.qr(rng.standard_normal((d, d)))
    lam = np.sort(rng.random(d) + 0.05)[::-1] * np.arange(d, 0, -1)
    X = np.sqrt(d) * np.sqrt(lam)[:, None] * q.T
    f = fit.fit_basis(X, fit.GAIN_ROTATE)
    assert np.allclose(f["lam"], lam, rtol=1e-10)
    # eigenvectors equal the columns of Q up to sign
    assert np.allclose(np.abs(f["U"].T @ q), np.eye(d), atol=1e-8)


def test_latent_second_moment_identity_eq4():
    """Eq. 4: with the square-root split the uncentred latent Y = X W_enc has Y^T Y / N = diag(sqrt(lam))."""
    X = _tiny_side(si.SIDE_K)
    f = fit.fit_basis(X, fit.GAIN_SQRT)
    Y = X @ f["W_enc"]
    S = Y.T @ Y / X.shape[0]
    target = np.sqrt(f["lam"])
    assert np.abs(S - np.diag(target)).max() <= 1e-9 * target[0]
    # centred variances and means are the measured ones
    Yc = Y - f["m_rot"][None, :]
    assert np.allclose(Yc.mean(axis=0), 0, atol=1e-9)
    assert np.allclose(Yc.var(axis=0), f["v_alloc"], rtol=1e-8, atol=1e-12)


def test_whitening_split_gives_unit_variance():
    X = _tiny_side(si.SIDE_V)
    f = fit.fit_basis(X, fit.GAIN_WHITEN)
    Yc = X @ f["W_enc"] - f["m_rot"][None, :]
    assert np.allclose(Yc.var(axis=0), 1.0, rtol=1e-8)


@pytest.mark.parametrize("mode", [fit.GAIN_ROTATE, fit.GAIN_SQRT, fit.GAIN_WHITEN])
def test_score_is_invariant_under_the_shared_rotation(mode):
    """q k^T = q' c^T with q' = W_dec q (appendix "Latent-space attention"), for every split of the spectrum."""
    X = _tiny_side(si.SIDE_K, 256)
    f = fit.fit_basis(X, mode)
    rng = np.random.default_rng(4)
    q = rng.standard_normal((5, X.shape[1]))
    c = X @ f["W_enc"]                        # uncentred latent = (y + m')
    qp = q @ f["W_dec"].T
    a = q @ X.T
    b = qp @ c.T
    assert np.abs(a - b).max() <= 1e-10 * np.abs(a).max()


def test_rotation_round_trip_through_fp32_matrices():
    X = _tiny_side(si.SIDE_K, 64)
    f = fit.fit_basis(_tiny_side(si.SIDE_K), fit.GAIN_SQRT)
    we, wd, mr = f["W_enc"].astype(np.float32), f["W_dec"].astype(np.float32), f["m_rot"].astype(np.float32)
    y = np.stack([codec.rotate_token(x, we, mr) for x in X.astype(np.float32)])
    # independent fp64 statement of the same product
    y_ref = X.astype(np.float32).astype(np.float64) @ we.astype(np.float64) - mr.astype(np.float64)
    assert np.abs(y - y_ref).max() <= 1e-6 * np.abs(y_ref).max()
    back = (y.astype(np.float64) + mr) @ wd.astype(np.float64)
    assert np.abs(back - X).max() <= 2e-5 * np.abs(X).max()


# ----------------------------------------------------------------------------- allocation

def test_allocation_worked_example_from_eq5():
    """v = [256, 16, 16, 1], mean rate 2: GM = 16, b = 2 + 0.5 log2(v / 16) = [4, 2, 2, 0]."""
    v = np.array([256.0, 16.0, 16.0, 1.0])
    assert np.allclose(fit.waterfill_closed_form(v, 2.0, 8), [4, 2, 2, 0])
    assert list(fit.alloc_bits(v, 8, b_max=8)) == [4, 2, 2, 0]


def test_allocation_matches_exhaustive_search():
    rng = np.random.default_rng(9)
    for _ in range(60):
        v = (rng.random(4) ** 3 * 100 + 1e-6).astype(np.float32)
        btot = int(rng.integers(0, 9))
        b = fit.alloc_bits(v, btot, b_max=4)
        assert b.sum() == min(btot, 16)
        best = min((sum(float(v[j]) * 4.0 ** -c[j] for j in range(4)))
                   for c in itertools.product(range(5), repeat=4) if sum(c) == min(btot, 16))
        got = sum(float(v[j]) * 4.0 ** -int(b[j]) for j in range(4))
        assert got <= best * (1 + 1e-12)


def test_allocation_structure_on_a_decaying_spectrum():
    d = 128
    v = (np.arange(1, d + 1) ** -1.5).astype(np.float32)
    for ratio in (4.0, 8.0, 12.0):
        btot = fit.total_bits(d, ratio)
        b = fit.alloc_bits(v, btot).astype(np.int64)
        assert b.sum() == btot and b.max() <= 8
        assert (np.diff(b) <= 0).all()                       # non-increasing along the energy order
        dist = v.astype(np.float64) * 4.0 ** -b
        # discrete water level: nobody below b_max would gain more from a bit than a holder would lose
        assert dist[b < 8].max() <= 4 * dist[b > 0].min() * (1 + 1e-12)
        # within one bit of the real-valued closed form (Eq. 5 with the clamp)
        closed = fit.waterfill_closed_form(v, btot / d, 8)
        inner = (closed > 0) & (closed < 8)
        assert np.abs(b - closed)[inner].max() < 1.0
    assert (fit.alloc_bits(v, fit.total_bits(d, 12.0)) == 0).any()   # the tail is dropped at low rate
    assert fit.total_bits(128, 12.0) == 170 and fit.total_bits(128, 4.0) == 512 and fit.total_bits(128, 8.0) == 256


def test_allocation_width_groups_and_clamp():
    v = (np.arange(1, 129) ** -2.0).astype(np.float32)
    b = fit.alloc_bits(v, 256, width_group=64)
    assert len(set(b[:64])) == 1 and len(set(b[64:])) == 1 and b.sum() == 256 and b[0] >= b[64]
    b = fit.alloc_bits(v, 256, width_group=2)
    assert (b[0::2] == b[1::2]).all() and b.sum() == 256
    assert list(fit.alloc_bits(np.ones(4), 100, b_max=8)) == [8, 8, 8, 8]
    assert list(fit.alloc_bits(np.array([1.0, 1.0, 1.0, 1.0]), 2)) == [1, 1, 0, 0]     # ties: lowest index first


# ----------------------------------------------------------------------------- rate accounting (paper's printed numbers)

def _golden_lines(kind):
    with open(os.path.join(GOLDEN, "paper_rate_accounting.txt")) as f:
        return [line.split()[1:] for line in f if line.startswith(kind + " ")]


def _printed(s):
    return float(s[:-1]) * (1e3 if s.endswith("k") else 1e6)


def test_effective_ratios_printed_in_the_paper():
    for bits, g, printed in _golden_lines("ratio"):
        widths = np.full(128, int(bits), np.uint8)
        r = fit.effective_ratio(widths, int(g))
        assert round(r, 2) == float(printed)
    # zero-bit groups store nothing, not even metadata
    w = np.zeros(128, np.uint8)
    w[:64] = 4
    assert fit.effective_bits_per_element(w, 64) == (64 * 4 + 32) / 128


def test_capacity_table_printed_in_the_paper():
    for layers, heads, hd, nbytes in _golden_lines("dense_bytes_per_token"):
        assert int(layers) * int(heads) * int(hd) * 2 * 2 == int(nbytes)     # K and V, 2 bytes each
    rows = _golden_lines("capacity")
    assert len(rows) == 20
    for budget, ratio, printed in rows:
        got = fit.max_context_tokens(float(budget), float(ratio))
        want = _printed(printed)
        digits = 3 if want >= 1e5 else 2           # the table prints 2-3 significant digits
        assert abs(got - want) <= 0.5 * 10 ** (np.floor(np.log10(want)) - digits + 1) * 1.0001


# ----------------------------------------------------------------------------- attention

def _coded_tiny(ratio=4.0, mode=fit.GAIN_SQRT, n=384, widths_override=None):
    wl = si.WORKLOADS["tiny"]
    out = {}
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        X = si.draw_unit(wl, 0, 0, side, 0)
        f = fit.fit_basis(X.astype(np.float64), mode)
        widths = fit.alloc_bits(f["v_alloc"], fit.total_bits(128, ratio)) if widths_override is None else \
            np.full(128, widths_override, np.uint8)
        tb = codec.tile_bytes(widths, 64)
        cache = np.zeros(((n + 127) // 128) * tb, np.uint8)
        we, wd, mr = (f[k].astype(np.float32) for k in ("W_enc", "W_dec", "m_rot"))
        st, _ = codec.encode_unit(X[:n], we, mr, widths, 64, side, 0, cache, tb)
        assert st == 0
        out[name] = dict(X=X[:n], widths=widths, tb=tb, cache=cache, we=we, wd=wd, mr=mr)
    return out


def _attend(c, q, mode, n):
    k, v = c["k"], c["v"]
    return codec.attention_units(mode, q[None], [n], k["cache"], [0], [k["tb"]], v["cache"], [0], [v["tb"]],
                                 k["wd"][None], k["mr"][None], k["widths"][None], v["wd"][None], v["mr"][None],
                                 v["widths"][None], 64, 1.0 / np.sqrt(128.0))


@pytest.mark.parametrize("mode", [fit.GAIN_ROTATE, fit.GAIN_SQRT, fit.GAIN_WHITEN])
def test_latent_attention_equals_reconstruct_then_attend(mode):
    n = 300                                      # ragged: two full tiles and a partial one
    c = _coded_tiny(4.0, mode, n)
    q = si.draw_queries(si.WORKLOADS["tiny"], 0, 0).astype(np.float64)
    oa, la = _attend(c, q, "A", n)
    ob, lb = _attend(c, q, "B", n)
    assert np.abs(oa - ob).max() <= 1e-10 * np.abs(oa).max()
    assert np.abs(la - lb).max() <= 1e-10


def _handworked_case():
    """Three tokens, d = 8, scale group 4, widths chosen so that every rotated coordinate lies exactly on its
    quantiser grid (group minimum, range and step are exact binary fractions): yhat = y with no rounding anywhere.
    Transforms are signed, scaled permutations (not involutions, so a transposed matrix changes the result) and
    the rotated means are as large as the data.  Everything below the inputs was worked out by hand."""
    d, gs = 8, 4
    k = dict(
        widths=np.array([2, 2, 2, 2, 1, 1, 0, 1], np.uint8),       # channel 6 is dropped: it reconstructs to its mean
        # group 0 (3 levels above the minimum): steps 1, 1, 0.25; group 1 (one bit): ranges 2, 1 and a constant group
        y=np.array([[-1.5, -0.5, 0.5, 1.5, 0, 2, 7.0, 2],
                    [1, -2, 0, -1, -1, 0, 7.0, -1],
                    [0.25, 1, 0.5, 0.75, 3, 3, 7.0, 3]], np.float32),
        m=np.array([0.5, -1, 2, 0, 1, 0, 3, -0.5], np.float32),
        perm=[2, 0, 3, 1, 6, 4, 7, 5], coef=[1, 2, -1, 0.5, 1, -2, 1, 4])
    v = dict(
        widths=np.array([2, 2, 0, 2, 1, 1, 1, 1], np.uint8),
        y=np.array([[2, -1, 9.0, 1, -4, -4, -2, -4],
                    [0, 0.75, 9.0, 0.25, 1, 1, 1, 1],
                    [-3, 3, 9.0, 1, 0.5, 1.5, 1.5, 0.5]], np.float32),
        m=np.array([-1, 0.5, 2, 1, 0, -2, 0.25, 4], np.float32),
        perm=[1, 3, 0, 2, 5, 7, 4, 6], coef=[2, 1, -1, 4, 0.5, 1, -2, 1])
    for side, c in ((codec.SIDE_K, k), (codec.SIDE_V, v)):
        w = np.zeros((d, d), np.float32)                            # xhat_i = coef_i * (yhat + m')_{perm_i}
        for i in range(d):
            w[c["perm"][i], i] = c["coef"][i]
        c["wd"] = w
        c["tb"] = codec.tile_bytes(c["widths"], gs)
        c["cache"] = np.zeros(c["tb"], np.uint8)
        st, _ = codec.encode_unit(c["y"], w, c["m"], c["widths"], gs, side, 0, c["cache"], c["tb"], rotated_input=True)
        assert st == 0
    # By hand: z = yhat + m' (dropped channel: z = m'), then xhat_i = coef_i * z_{perm_i}
    k_hat = np.array([[2.5, -2.0, -1.5, -0.75, 3.0, -2.0, 1.5, 8.0],
                      [2.0, 3.0, 1.0, -1.5, 3.0, 0.0, -1.5, 0.0],
                      [2.5, 1.5, -0.75, 0.0, 3.0, -8.0, 2.5, 12.0]])
    v_hat = np.array([[-1.0, 2.0, -1.0, 8.0, -3.0, 0.0, 8.0, -1.75],
                      [2.5, 1.25, 1.0, 8.0, -0.5, 5.0, -2.0, 1.25],
                      [7.0, 2.0, 4.0, 8.0, -0.25, 4.5, -1.0, 1.75]])
    return d, gs, k, v, k_hat, v_hat


@pytest.mark.parametrize("mode", ["A", "B"])
def test_attention_on_a_handworked_case(mode):
    """Sec. 3.3 (Mode A: reconstruct, then attend) and the appendix "Latent-space attention and memory" (Mode B:
    q' = q W_up^T, scores q' c^T, one lift of the output) on a case small enough to work by hand, with rotated
    means m'_K, m'_V that matter, a dropped channel and a constant group.  Head 0 has q = 0: every score is equal,
    the output is the plain mean of the three reconstructed values and lse = ln 3.  Head 1: the three scores
    scale * q . k_hat_t are 0.125, -0.625 and -0.4375."""
    d, gs, k, v, k_hat, v_hat = _handworked_case()
    _, xk = codec.decode_unit(k["cache"], k["tb"], 3, k["wd"], k["m"], k["widths"], gs, codec.SIDE_K)
    _, xv = codec.decode_unit(v["cache"], v["tb"], 3, v["wd"], v["m"], v["widths"], gs, codec.SIDE_V)
    assert np.array_equal(xk, k_hat) and np.array_equal(xv, v_hat)
    q = np.array([[0.0] * 8, [0.5, -0.25, 0, 1, 0, 0.125, 0, -0.0625]])
    out, lse = codec.attention_units(mode, q[None], [3], k["cache"], [0], [k["tb"]], v["cache"], [0], [v["tb"]],
                                     k["wd"][None], k["m"][None], k["widths"][None], v["wd"][None], v["m"][None],
                                     v["widths"][None], gs, 0.5)
    mean_v = [(-1.0 + 2.5 + 7.0) / 3, (2.0 + 1.25 + 2.0) / 3, (-1.0 + 1.0 + 4.0) / 3, 8.0, (-3.0 - 0.5 - 0.25) / 3,
              (0.0 + 5.0 + 4.5) / 3, (8.0 - 2.0 - 1.0) / 3, (-1.75 + 1.25 + 1.75) / 3]
    assert np.abs(out[0, 0] - mean_v).max() <= 1e-14
    assert abs(lse[0, 0] - math.log(3.0)) <= 1e-14
    e = [math.exp(0.125), math.exp(-0.625), math.exp(-0.4375)]
    want = [(e[0] * v_hat[0][i] + e[1] * v_hat[1][i] + e[2] * v_hat[2][i]) / sum(e) for i in range(8)]
    assert np.abs(out[0, 1] - want).max() <= 1e-14
    assert abs(lse[0, 1] - math.log(sum(e))) <= 1e-14
    # one token fewer is a different answer: the functions attend to exactly n tokens
    out2, _ = codec.attention_units(mode, q[None], [2], k["cache"], [0], [k["tb"]], v["cache"], [0], [v["tb"]],
                                    k["wd"][None], k["m"][None], k["widths"][None], v["wd"][None], v["m"][None],
                                    v["widths"][None], gs, 0.5)
    assert np.abs(out2[0, 0] - (v_hat[0] + v_hat[1]) / 2).max() <= 1e-14


def test_attention_at_eight_bits_is_within_the_quantisation_bound_of_dense_attention():
    """Mode A at 8 bits per channel against textbook softmax attention on the raw vectors.  The tolerance is the
    bound the quantisation error itself gives: with delta = max_t |scale q.(k_hat_t - k_t)| the softmax weights
    move by at most e^(2 delta) - 1 in total variation, so
        |out - dense| <= max_t |v_hat_t - v_t|_inf + (e^(2 delta) - 1) max_t |v_t|_inf,   |lse - lse_dense| <= delta."""
    n = 256
    c = _coded_tiny(4.0, fit.GAIN_WHITEN, n, widths_override=8)
    q = si.draw_queries(si.WORKLOADS["tiny"], 0, 0).astype(np.float64)
    oa, la = _attend(c, q, "A", n)
    K, V = c["k"]["X"].astype(np.float64), c["v"]["X"].astype(np.float64)
    k, v = c["k"], c["v"]
    _, k_hat = codec.decode_unit(k["cache"], k["tb"], n, k["wd"], k["mr"], k["widths"], 64, codec.SIDE_K)
    _, v_hat = codec.decode_unit(v["cache"], v["tb"], n, v["wd"], v["mr"], v["widths"], 64, codec.SIDE_V)
    scale = 1.0 / np.sqrt(128.0)
    s = q @ K.T * scale
    p = np.exp(s - s.max(axis=1, keepdims=True))
    lse = np.log(p.sum(axis=1)) + s.max(axis=1)
    p /= p.sum(axis=1, keepdims=True)
    assert np.allclose(p.sum(axis=1), 1.0)
    dense = p @ V
    delta = np.abs(q @ (k_hat - K).T * scale).max(axis=1)                    # per head
    bound = np.abs(v_hat - V).max() + (np.exp(2 * delta) - 1) * np.abs(V).max()
    assert delta.max() < 0.02 and bound.max() < 0.03      # an order of magnitude below the tolerances this replaces
    assert (np.abs(oa[0] - dense).max(axis=1) <= bound * (1 + 1e-9)).all()
    assert (np.abs(la[0] - lse) <= delta * (1 + 1e-9)).all()


def test_reconstruction_error_shrinks_with_rate_and_respects_step():
    errs = []
    for ratio in (12.0, 8.0, 4.0):
        c = _coded_tiny(ratio, fit.GAIN_SQRT, 256)
        k = c["k"]
        _, xhat = codec.decode_unit(k["cache"], k["tb"], 256, k["wd"], k["mr"], k["widths"], 64, codec.SIDE_K)
        errs.append(np.linalg.norm(xhat - k["X"]) / np.linalg.norm(k["X"]))
    assert errs[0] > errs[1] > errs[2]
    assert errs[2] < 0.1


def test_importance_allocation_beats_uniform_at_low_rate():
    """Observation 2, qualitatively: at 2 bits per channel, water-filled widths give a lower attention-output
    error than uniform widths on the same data."""
    n = 384
    q = si.draw_queries(si.WORKLOADS["tiny"], 0, 0).astype(np.float64)
    dense = _attend(_coded_tiny(4.0, fit.GAIN_WHITEN, n, widths_override=8), q, "A", n)[0]
    wf = _attend(_coded_tiny(8.0, fit.GAIN_WHITEN, n), q, "A", n)[0]
    un = _attend(_coded_tiny(8.0, fit.GAIN_WHITEN, n, widths_override=2), q, "A", n)[0]
    assert np.linalg.norm(wf - dense) < np.linalg.norm(un - dense)


# ----------------------------------------------------------------------------- pooled allocation, key/value split

def _objective(v, b):
    return float((np.asarray(v, np.float64) * 4.0 ** (-np.asarray(b, np.float64))).sum())


def test_pooled_allocation_is_the_optimum_over_all_heads_together():
    """Sec. 3.2 with the latent spanning all KV heads (appendix, bit-profile figure): the pooled allocation spends
    exactly the pooled budget, never does worse than allocating head by head, equals it when the heads are
    identical, moves bits from a weak head to a strong one, and still satisfies the discrete water level
    D_i <= 4 D_j across heads (equal slope, Eq. 5)."""
    rng = np.random.default_rng(5)
    d, H, btot = 128, 4, 256
    base = ((np.arange(1, d + 1) ** -1.5) * rng.uniform(0.9, 1.1, d)).astype(np.float32)   # no exact ties
    same = np.stack([base] * H)
    pooled = fit.alloc_bits_pooled(same, btot)
    assert np.array_equal(pooled, np.stack([fit.alloc_bits(base, btot)] * H))
    scales = np.array([4.0, 1.0, 0.25, 0.01], np.float32)
    v = base[None] * scales[:, None] * rng.uniform(0.9, 1.1, (H, d)).astype(np.float32)
    pooled = fit.alloc_bits_pooled(v, btot)
    single = np.stack([fit.alloc_bits(v[h], btot) for h in range(H)])
    assert pooled.sum() == H * btot == single.sum()
    assert _objective(v, pooled) <= _objective(v, single)
    per_head = pooled.sum(axis=1)
    assert per_head[0] > per_head[1] > per_head[2] > per_head[3]
    D = v.astype(np.float64) * 4.0 ** (-pooled.astype(np.float64))
    assert D[pooled < 8].max() <= 4.0 * D[pooled > 0].min() * (1 + 1e-12)
    # brute force on a tiny pool: 2 heads x 3 channels, 5 bits, widths up to 3
    import itertools
    vt = np.array([[9.0, 1.0, 0.1], [30.0, 0.5, 0.4]], np.float32)
    got = fit.alloc_bits_pooled(vt, 5 // 2 + 0, b_max=3)          # 2 bits per head: 4 in the pool
    best = min((b for b in itertools.product(range(4), repeat=6) if sum(b) == 4),
               key=lambda b: _objective(vt.reshape(-1), b))
    assert _objective(vt.reshape(-1), got.reshape(-1)) == _objective(vt.reshape(-1), best)
    # one width per group of 64 coordinates, pooled over 8 heads: 16 groups compete (the paper's structure)
    v8 = base[None] * rng.uniform(0.05, 3.0, (8, 1)).astype(np.float32)
    g = fit.alloc_bits_pooled(v8, 256, width_group=64)
    assert g.sum() == 8 * 256 and all(len(set(row[:64])) == 1 and len(set(row[64:])) == 1 for row in g)


def test_key_value_budget_split():
    """Sec. 3.1 (last paragraph): the keys get the fraction kappa of the joint budget.  kappa = 1/2 leaves both sides
    at the nominal ratio; for any kappa the two budgets add up to the joint one."""
    assert fit.split_ratio(8.0, 0.5) == (8.0, 8.0)
    for kappa in (0.25, 0.4, 0.75):
        rk, rv = fit.split_ratio(8.0, kappa)
        bits_k, bits_v = 16 * 128 / rk, 16 * 128 / rv
        assert abs(bits_k + bits_v - 2 * 16 * 128 / 8.0) < 1e-9
        assert abs(bits_k / (bits_k + bits_v) - kappa) < 1e-12


# ----------------------------------------------------------------------------- rotary position embedding

def test_rope_rows_against_closed_forms():
    """The position rotation of Sec. 3.3 (applied to the reconstructed key): position 0 is the identity; d = 4 at
    position 1 with theta = 10000 rotates the pair (x0, x2) by 1 rad and (x1, x3) by 0.01 rad (hand values); norms are
    kept; and (R(a) q) . (R(b) k) depends on a - b only."""
    x = np.array([[1.0, 2.0, 3.0, 4.0]])
    assert np.array_equal(codec.rope_rows(x, 0, 10000.0), x)
    y = codec.rope_rows(np.array([[1.0, 2.0, 3.0, 4.0], [1.0, 2.0, 3.0, 4.0]]), 0, 10000.0)[1]
    want = [1 * math.cos(1.0) - 3 * math.sin(1.0), 2 * math.cos(0.01) - 4 * math.sin(0.01),
            3 * math.cos(1.0) + 1 * math.sin(1.0), 4 * math.cos(0.01) + 2 * math.sin(0.01)]
    assert np.abs(y - want).max() <= 1e-15
    rng = np.random.default_rng(2)
    q, k = rng.standard_normal((1, 128)), rng.standard_normal((1, 128))
    for a, b in ((5, 3), (1005, 1003), (77, 75)):
        ra = codec.rope_rows(q, a, 500000.0)[0]
        rb = codec.rope_rows(k, b, 500000.0)[0]
        assert abs(np.linalg.norm(ra) - np.linalg.norm(q)) <= 1e-12
        if a == 5:
            first = ra @ rb
        assert abs(ra @ rb - first) <= 1e-9


@pytest.mark.parametrize("gain_mode", [fit.GAIN_SQRT, fit.GAIN_WHITEN])
def test_rope_latent_attention_equals_reconstruct_rotate_attend(gain_mode):
    """With RoPE, Mode A (reconstruct the key, rotate it at its position, attend: Sec. 3.3) and the latent-space form
    (rotate the query back per token and fold it through W_dec,K: the appendix's q' with the position rotation moved
    to the query side) agree to 1e-10; without positions (theta large, all angles ~ 0 at pos0 = 0 for a tiny n) both
    fall back to the plain functions; and the rotated reconstruction equals the rotation of the plain one."""
    n = 200
    c = _coded_tiny(6.0, gain_mode, n)
    k, v = c["k"], c["v"]
    q = si.draw_queries(si.WORKLOADS["tiny"], 0, 0).astype(np.float64)
    theta, pos0 = 500000.0, 1234.0
    q_rot = np.stack([codec.rope_rows(q[h][None], pos0 + n, theta)[0] for h in range(q.shape[0])])
    args = (n, k["cache"], k["tb"], v["cache"], v["tb"], k["wd"], k["mr"], k["widths"], v["wd"], v["mr"], v["widths"], 64,
            1.0 / np.sqrt(128.0), pos0, theta)
    oa, la = codec.attention_rope_unit("A", q_rot, *args)
    ob, lb = codec.attention_rope_unit("B", q_rot, *args)
    assert np.abs(oa - ob).max() <= 1e-10 * np.abs(oa).max() and np.abs(la - lb).max() <= 1e-10
    # the rotated reconstruction = rotation of the plain reconstruction; a dense check of Mode A on top of it
    _, k_hat = codec.decode_unit(k["cache"], k["tb"], n, k["wd"], k["mr"], k["widths"], 64, codec.SIDE_K)
    _, v_hat = codec.decode_unit(v["cache"], v["tb"], n, v["wd"], v["mr"], v["widths"], 64, codec.SIDE_V)
    k_rot = codec.decode_unit_rope(k["cache"], k["tb"], n, k["wd"], k["mr"], k["widths"], 64, codec.SIDE_K, pos0, theta)
    assert np.abs(k_rot - codec.rope_rows(k_hat, pos0, theta)).max() == 0.0
    s = q_rot @ k_rot.T / np.sqrt(128.0)
    p = np.exp(s - s.max(axis=1, keepdims=True))
    p /= p.sum(axis=1, keepdims=True)
    assert np.abs(oa - p @ v_hat).max() <= 1e-12 * np.abs(oa).max()
    # relative positions only: shifting every position (query included) by the same amount changes nothing
    q_rot2 = np.stack([codec.rope_rows(q[h][None], pos0 + 977 + n, theta)[0] for h in range(q.shape[0])])
    oa2, _ = codec.attention_rope_unit("A", q_rot2, *args[:-2], pos0 + 977, theta)
    assert np.abs(oa2 - oa).max() <= 1e-9 * np.abs(oa).max()
    # and with all angles zero (position 0 only matters through pos * theta^..: use n = 1 at pos0 = 0)
    o1, l1 = codec.attention_rope_unit("B", q, 1, *args[1:-2], 0.0, theta)
    o0, l0 = codec.attention_units("B", q[None], [1], k["cache"], [0], [k["tb"]], v["cache"], [0], [v["tb"]],
                                   k["wd"][None], k["mr"][None], k["widths"][None], v["wd"][None], v["mr"][None],
                                   v["widths"][None], 64, 1.0 / np.sqrt(128.0))
    assert np.abs(o1 - o0[0]).max() <= 1e-13 and np.abs(l1 - l0[0]).max() <= 1e-13


# ---------------------------------------------------------------- many-query (prefill) attention, Mode A
def test_prefill_on_the_handworked_case():
    """Sec. 3.3, Mode A with a chunk of queries: query i sits at position pos0 + i and attends tokens 0 .. pos0 + i.
    On the hand-worked cache (three tokens, pos0 = 1, two new queries): the first query sees two tokens, the second
    all three.  With q = 0 the outputs are the plain means of the reconstructed values it may see; the second head
    repeats the single-query case's scores 0.125, -0.625, -0.4375."""
    from oracle import prefill
    d, gs, k, v, k_hat, v_hat = _handworked_case()
    q1 = [0.5, -0.25, 0, 1, 0, 0.125, 0, -0.0625]
    q = np.array([[[0.0] * 8, q1], [[0.0] * 8, q1]])              # [n_new = 2, G = 2, d]
    out, lse = prefill.prefill_mode_a(q, 1, k["cache"], k["tb"], v["cache"], v["tb"], k["wd"], k["m"], k["widths"],
                                      v["wd"], v["m"], v["widths"], gs, 0.5)
    assert np.abs(out[0, 0] - (v_hat[0] + v_hat[1]) / 2).max() <= 1e-14 and abs(lse[0, 0] - math.log(2.0)) <= 1e-14
    assert np.abs(out[1, 0] - (v_hat[0] + v_hat[1] + v_hat[2]) / 3).max() <= 1e-14
    e = [math.exp(0.125), math.exp(-0.625), math.exp(-0.4375)]
    want0 = (e[0] * v_hat[0] + e[1] * v_hat[1]) / (e[0] + e[1])
    want1 = (e[0] * v_hat[0] + e[1] * v_hat[1] + e[2] * v_hat[2]) / sum(e)
    assert np.abs(out[0, 1] - want0).max() <= 1e-14 and abs(lse[0, 1] - math.log(e[0] + e[1])) <= 1e-14
    assert np.abs(out[1, 1] - want1).max() <= 1e-14 and abs(lse[1, 1] - math.log(sum(e))) <= 1e-14


def test_prefill_rows_equal_single_query_attention_at_their_lengths():
    """Row i of the chunked computation is the single-query Mode A attention (the C oracle, pinned above) over the
    first pos0 + i + 1 tokens: the causal limit is per row, off by one in neither direction."""
    from oracle import prefill
    n, pos0 = 300, 250
    c = _coded_tiny(4.0, fit.GAIN_SQRT, n)
    k, v = c["k"], c["v"]
    rng = np.random.default_rng(5)
    q = rng.standard_normal((n - pos0, 4, 128))
    scale = 1.0 / np.sqrt(128.0)
    out, lse = prefill.prefill_mode_a(q, pos0, k["cache"], k["tb"], v["cache"], v["tb"], k["wd"], k["mr"], k["widths"],
                                      v["wd"], v["mr"], v["widths"], 64, scale)
    for i in (0, 1, 5, 6, 49):                                     # 256 tokens (a tile edge) is row 5
        oa, la = _attend(c, q[i], "A", pos0 + i + 1)
        assert np.abs(out[i] - oa[0]).max() <= 1e-12 * max(1.0, np.abs(oa).max())
        assert np.abs(lse[i] - la[0]).max() <= 1e-12


def test_bf16_rounding_helper():
    """Round to nearest, ties to even, on the 16 bits below bfloat16's mantissa."""
    from oracle import prefill
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -7, 1.0 + 3 * 2.0 ** -8, -(1.0 + 2.0 ** -8 + 2.0 ** -20), 0.0,
                  3.0e-5])
    r = prefill.round_bf16(x)
    # halfway cases go to the even mantissa: 1 + 2^-8 -> 1, 1 + 3 * 2^-8 -> 1 + 2^-6; just above halfway rounds away
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2.0 ** -7 and r[3] == 1.0 + 2.0 ** -6
    assert r[4] == -(1.0 + 2.0 ** -7) and r[5] == 0.0
    assert abs(r[6] - 3.0e-5) <= 3.0e-5 * 2.0 ** -9
