"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded inputs.

Bars (from the benchmark spec): codes, widths and packed bytes bit-exact when both sides start from the
same rotated fp32 coordinates; end to end only +-1-level rounding ties in at most 1e-4 of the entries;
reconstructions and attention outputs within 2e-3 (max |diff| / max |oracle| per vector).
"""
import dataclasses

import numpy as np
import pytest

import spectra_inputs as si
from oracle import codec as oc
from oracle import fit as ofit
from tests import helpers as H

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 2e-3
MISMATCH_RATE = 1e-4


@pytest.fixture(scope="module")
def sp():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2608_07915_b200 as sp
    sp.lib()
    return sp


def _sync_status(status):
    torch.cuda.synchronize()
    return int(status.item())


def _gpu_encode(sp, cfg, params, dp, side, x_units, pos0, cache_dev, off_dev, rotated=False):
    n_units, n_new, d = x_units.shape
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sp.encode(cfg, side, x_units, sp.ROTATED_INPUT if rotated else 0, n_units, params.n_sets, pos0, n_new,
              n_new * d, d, dp["w_enc"], dp["m_rot"], dp["widths"], cache_dev, off_dev, status)
    return _sync_status(status)


# ----------------------------------------------------------------------------- allocation

@pytest.mark.parametrize("width_group", [1, 2, 64])
def test_alloc_bits_is_bit_exact(sp, width_group):
    rng = np.random.default_rng(100 + width_group)
    n_units = 37
    v = (rng.random((n_units, 128)) ** 6 * 10.0 ** rng.integers(-3, 3, (n_units, 1))).astype(np.float32)
    v[3] = np.sort(v[3])[::-1]
    v[5, 40:] = 0.0                                            # dead tail
    v[7] = 1.0                                                 # all ties
    cfg = sp.default_config(width_group=width_group)
    for ratio in (4.0, 8.0, 12.0, 1.5):
        widths = torch.zeros((n_units, 128), dtype=torch.uint8, device="cuda")
        sp.alloc_bits(cfg, H.to_dev(v), n_units, ratio, widths)
        got = widths.cpu().numpy()
        btot = sp.total_bits(cfg, ratio)
        assert btot == min(ofit.total_bits(128, ratio), 8 * 128)
        for u in range(n_units):
            want = ofit.alloc_bits(v[u], btot, 8, width_group)
            assert np.array_equal(got[u], want), (ratio, u)


# ----------------------------------------------------------------------------- encode from rotated inputs

def _random_widths(rng, kind):
    if kind == "mixed":
        return rng.integers(0, 9, 128).astype(np.uint8)
    if kind == "dead_group":
        w = rng.integers(0, 5, 128).astype(np.uint8)
        w[64:] = 0
        return w
    if kind == "odd_classes":
        w = np.zeros(128, np.uint8)
        w[:7] = [7, 5, 3, 1, 8, 6, 2]                          # odd strip counts in several classes
        return w
    return np.full(128, int(kind), np.uint8)


@pytest.mark.parametrize("kind", ["mixed", "dead_group", "odd_classes", "8", "1", "3"])
@pytest.mark.parametrize("gs", [64, 32, 128])
def test_encode_from_rotated_inputs_is_bit_exact(sp, kind, gs):
    if gs != 64 and kind not in ("mixed", "dead_group"):
        pytest.skip("scale-group variants run on two width patterns only")
    rng = np.random.default_rng(7)
    n_units, n = 3, 300                                        # two full tiles and a ragged third
    widths = np.stack([_random_widths(rng, kind) for _ in range(n_units)])
    eye = np.tile(np.eye(128, dtype=np.float32), (n_units, 1, 1))
    params = H.Params(eye, eye, np.zeros((n_units, 128)), widths, gs)
    y = (rng.standard_normal((n_units, n, 128)) * 10.0 ** rng.integers(-2, 3, (n_units, 1, 128))).astype(np.float32)
    y[0, 5] = 1.25                                             # a constant token: zero range
    cfg = sp.default_config(scale_group=gs)
    for side in (sp.SIDE_K, sp.SIDE_V):
        off, total = H.cache_layout(params, n_units, n)
        ref = np.zeros(total, np.uint8)
        assert H.oracle_encode(params, side, y, np.zeros(n_units, np.int64), ref, off, rotated=True) == 0
        cache = torch.full((total,), 0xAA, dtype=torch.uint8, device="cuda")      # dirty buffer on purpose
        pos0 = torch.zeros(n_units, dtype=torch.int32, device="cuda")
        st = _gpu_encode(sp, cfg, params, H.dev_params(params), side, H.to_dev(y), pos0, cache, H.to_dev(off),
                         rotated=True)
        assert st == 0
        got = cache.cpu().numpy()
        for u in range(n_units):
            tb = int(params.tile_bytes[u])
            assert sp.tile_bytes(cfg, widths[u]) == tb
            a, b = off[u], off[u] + 3 * tb
            assert np.array_equal(got[a:b], ref[a:b]), (side, u)


def test_encode_appends_preserve_earlier_tokens(sp):
    rng = np.random.default_rng(8)
    n_units = 2
    widths = np.stack([_random_widths(rng, "mixed") for _ in range(n_units)])
    eye = np.tile(np.eye(128, dtype=np.float32), (n_units, 1, 1))
    params = H.Params(eye, eye, np.zeros((n_units, 128)), widths, 64)
    y = rng.standard_normal((n_units, 400, 128)).astype(np.float32)
    cfg = sp.default_config()
    dp = H.dev_params(params)
    for side in (sp.SIDE_K, sp.SIDE_V):
        off, total = H.cache_layout(params, n_units, 400)
        ref = np.zeros(total, np.uint8)
        H.oracle_encode(params, side, y, np.zeros(n_units, np.int64), ref, off, rotated=True)
        cache = torch.full((total,), 0x55, dtype=torch.uint8, device="cuda")
        pos = 0
        for chunk in (100, 1, 1, 27, 150, 120, 1):             # crosses tile boundaries at odd places
            pos0 = torch.full((n_units,), pos, dtype=torch.int32, device="cuda")
            st = _gpu_encode(sp, cfg, params, dp, side, H.to_dev(y[:, pos:pos + chunk]), pos0, cache, H.to_dev(off),
                             rotated=True)
            assert st == 0
            pos += chunk
        assert pos == 400
        got = cache.cpu().numpy()
        for u in range(n_units):
            tb = int(params.tile_bytes[u])
            assert np.array_equal(got[off[u]:off[u] + 4 * tb], ref[off[u]:off[u] + 4 * tb])


def test_encode_per_unit_positions_and_status_bits(sp):
    rng = np.random.default_rng(9)
    widths = np.stack([_random_widths(rng, "4")] * 2)
    eye = np.tile(np.eye(128, dtype=np.float32), (2, 1, 1))
    params = H.Params(eye, eye, np.zeros((2, 128)), widths, 64)
    cfg = sp.default_config()
    y = rng.standard_normal((2, 3, 128)).astype(np.float32)
    off, total = H.cache_layout(params, 2, 256)
    ref = np.zeros(total, np.uint8)
    pos0 = np.array([5, 130], np.int64)
    H.oracle_encode(params, sp.SIDE_K, y, pos0, ref, off, rotated=True)
    cache = torch.zeros(total, dtype=torch.uint8, device="cuda")
    st = _gpu_encode(sp, cfg, params, H.dev_params(params), sp.SIDE_K, H.to_dev(y), H.to_dev(pos0.astype(np.int32)),
                     cache, H.to_dev(off), rotated=True)
    assert st == 0 and np.array_equal(cache.cpu().numpy(), ref)
    bad = y.copy()
    bad[0, 1, 3] = np.nan
    bad[1, 0, 7] = 1e9
    st = _gpu_encode(sp, cfg, params, H.dev_params(params), sp.SIDE_K, H.to_dev(bad), H.to_dev(pos0.astype(np.int32)),
                     cache, H.to_dev(off), rotated=True)
    assert st == (sp.STATUS_NONFINITE | sp.STATUS_F16_RANGE)


def test_bulk_bf16_encode_with_ragged_starts_keeps_earlier_tokens(sp):
    """The bulk bf16 path (rotation on tcgen05) on ranges that start and end inside tiles, different per unit, on
    top of tokens written before: earlier tokens stay byte for byte, the new ones match the oracle's encode of the
    same bf16 vectors up to rare rounding ties, slots behind the range are cleared."""
    wl = si.WORKLOADS["tiny"]
    cfg = sp.default_config()
    n_units, cap = 2, 640
    X = [si.to_bf16_f32(si.draw_unit(wl, 0, u, si.SIDE_K, 0)[:cap]) for u in range(n_units)]
    params = H.fit_params(X, 8.0)
    dp = H.dev_params(params)
    off, total = H.cache_layout(params, n_units, cap)
    first = np.array([70, 129], np.int64)            # tokens [0, first) are written beforehand, one by one path aside
    n_new = 300                                      # ends at 370 and 429: inside tiles
    for side in (sp.SIDE_K, sp.SIDE_V):
        ref = np.zeros(total, np.uint8)
        cache = torch.zeros(total, dtype=torch.uint8, device="cuda")
        for u in range(n_units):                     # the earlier tokens, by the oracle on both sides
            H.oracle_encode(H.Params(params.w_enc[[u]], params.w_dec[[u]], params.m_rot[[u]], params.widths[[u]], 64),
                            side, X[u][None, :first[u]], [0], ref[off[u]:], np.zeros(1, np.int64))
        cache.copy_(torch.from_numpy(ref))
        before = ref.copy()
        xs = np.stack([X[u][first[u]:first[u] + n_new] for u in range(n_units)])
        assert H.oracle_encode(params, side, xs, first, ref, off) == 0
        st = _gpu_encode(sp, cfg, params, dp, side, H.to_dev(xs).to(torch.bfloat16),
                         H.to_dev(first.astype(np.int32)), cache, H.to_dev(off))
        assert st == 0
        got = cache.cpu().numpy()
        for u in range(n_units):
            end = int(first[u]) + n_new
            c_ref, m_ref = H.unpack_codes(params, side, ref, off, u, end)
            c_got, m_got = H.unpack_codes(params, side, got, off, u, end)
            c_old, m_old = H.unpack_codes(params, side, before, off, u, int(first[u]))
            assert np.array_equal(c_got[:first[u]], c_old) and np.array_equal(m_got[:first[u]], m_old)
            # all tokens alike: codes within one level (a handful of ties in 300 tokens x 128 channels), metadata within
            # one fp16 step
            diff = np.abs(c_got.astype(np.int64) - c_ref.astype(np.int64))
            assert diff.max() <= 1 and (diff != 0).sum() <= 3
            meta = np.abs(H.f16_ordinal(m_got) - H.f16_ordinal(m_ref))
            assert meta.max() <= 1 and (meta.max(axis=1) != 0).sum() <= 3
            # slots of the last touched tile behind the range hold zeros
            tail_tile_end = (end + 127) // 128 * 128
            c_tail, m_tail = H.unpack_codes(params, side, got, off, u, tail_tile_end)
            assert not c_tail[end:].any() and not m_tail[end:].any()


@pytest.mark.parametrize("kind", ["mixed", "dead_group", "odd_classes", "8", "7", "1", "3"])
def test_bulk_bf16_encode_on_every_width_profile(sp, kind):
    """The bulk bf16 path (rotation on tcgen05, channel-major code tile, gathered half-words) on width profiles that
    use every class, every sub-field shift, classes with an odd number of strips and an empty scale group: whole and
    partly filled tiles, both sides, against the oracle's encode of the same bf16 vectors up to rare rounding ties."""
    wl = si.WORKLOADS["tiny"]
    cfg = sp.default_config()
    rng = np.random.default_rng(23)
    n = 300                                               # two whole tiles and a ragged one
    X = si.to_bf16_f32(si.draw_unit(wl, 0, 0, si.SIDE_K, 0)[:n])
    params = H.fit_params([X], 4.0, widths_override=_random_widths(rng, kind))
    dp = H.dev_params(params)
    off, total = H.cache_layout(params, 1, n)
    zero = np.zeros(1, np.int64)
    for side in (sp.SIDE_K, sp.SIDE_V):
        ref = np.zeros(total, np.uint8)
        assert H.oracle_encode(params, side, X[None], zero, ref, off) == 0
        cache = torch.zeros(total, dtype=torch.uint8, device="cuda")
        st = _gpu_encode(sp, cfg, params, dp, side, H.to_dev(X[None]).to(torch.bfloat16), H.to_dev(zero.astype(np.int32)),
                         cache, H.to_dev(off))
        assert st == 0
        got = cache.cpu().numpy()
        c_ref, m_ref = H.unpack_codes(params, side, ref, off, 0, n)
        c_got, m_got = H.unpack_codes(params, side, got, off, 0, n)
        diff = np.abs(c_got.astype(np.int64) - c_ref.astype(np.int64))
        assert diff.max() <= 1 and (diff != 0).sum() <= 6
        meta = np.abs(H.f16_ordinal(m_got) - H.f16_ordinal(m_ref))
        assert meta.max() <= 1 and (meta.max(axis=1) != 0).sum() <= 3
        # where codes and metadata agree the bytes do too: a token-wise comparison of the packed tiles' unpacked
        # content is the whole content, so nothing else may differ
        tb = int(params.tile_bytes[0])
        same_tiles = [t for t in range((n + 127) // 128)
                      if not diff[t * 128:(t + 1) * 128].any() and not meta[t * 128:(t + 1) * 128].any()]
        for t in same_tiles:
            assert np.array_equal(got[off[0] + t * tb: off[0] + (t + 1) * tb], ref[off[0] + t * tb: off[0] + (t + 1) * tb])


def test_bulk_bf16_encode_with_a_nan_and_an_out_of_range_token(sp):
    """The bulk bf16 path on whole tiles with one token that holds a NaN and one whose rotated values leave fp16's
    range: both are reported in the status word, every other token is stored exactly as without them, and the
    out-of-range token is stored with its offset and range clipped and its codes saturated, as the oracle stores it."""
    wl = si.WORKLOADS["tiny"]
    cfg = sp.default_config()
    n_units, n = 2, 512
    X = [si.to_bf16_f32(si.draw_unit(wl, 0, u, si.SIDE_K, 0)[:n]) for u in range(n_units)]
    params = H.fit_params(X, 8.0)
    dp = H.dev_params(params)
    off, total = H.cache_layout(params, n_units, n)
    clean = np.stack(X)
    bad = clean.copy()
    bad[0, 130, 5] = np.nan
    bad[1, 300] = si.to_bf16_f32(bad[1, 300] * 3.0e6)
    zero = np.zeros(n_units, np.int64)
    for side in (sp.SIDE_K, sp.SIDE_V):
        caches = []
        for x, want in ((clean, 0), (bad, sp.STATUS_NONFINITE | sp.STATUS_F16_RANGE)):
            cache = torch.zeros(total, dtype=torch.uint8, device="cuda")
            st = _gpu_encode(sp, cfg, params, dp, side, H.to_dev(x).to(torch.bfloat16), H.to_dev(zero.astype(np.int32)),
                             cache, H.to_dev(off))
            assert st == want
            caches.append(cache.cpu().numpy())
        ref = np.zeros(total, np.uint8)
        assert H.oracle_encode(params, side, bad[:, :, :], zero, ref, off) == (sp.STATUS_NONFINITE | sp.STATUS_F16_RANGE)
        for u, t_bad in ((0, 130), (1, 300)):
            c0, m0 = H.unpack_codes(params, side, caches[0], off, u, n)
            c1, m1 = H.unpack_codes(params, side, caches[1], off, u, n)
            keep = np.arange(n) != t_bad
            assert np.array_equal(c0[keep], c1[keep]) and np.array_equal(m0[keep], m1[keep])
        c_ref, m_ref = H.unpack_codes(params, side, ref, off, 1, n)
        c_got, m_got = H.unpack_codes(params, side, caches[1], off, 1, n)
        assert np.abs(c_got[300].astype(np.int64) - c_ref[300].astype(np.int64)).max() <= 1
        assert np.abs(H.f16_ordinal(m_got[300]) - H.f16_ordinal(m_ref[300])).max() <= 1
        assert c_got[300].max() > 0                        # the token is stored, not dropped


# ----------------------------------------------------------------------------- config 0 end to end

def _tiny_setup(sp, ratio=4.0, gain_mode=ofit.GAIN_SQRT, n=1024, gs=64):
    wl = si.WORKLOADS["tiny"]
    out = {}
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        X = si.draw_unit(wl, 0, 0, side, 0)
        params = H.fit_params([X], ratio, gs=gs, gain_mode=gain_mode)
        off, total = H.cache_layout(params, 1, n)
        out[name] = dict(X=X[:n], params=params, off=off, total=total)
    return wl, out


@pytest.mark.parametrize("gain_mode", [ofit.GAIN_ROTATE, ofit.GAIN_SQRT, ofit.GAIN_WHITEN])
def test_tiny_encode_end_to_end_mismatches_are_rare_ties(sp, gain_mode):
    wl, S = _tiny_setup(sp, 4.0, gain_mode)
    cfg = sp.default_config()
    for side, name in ((sp.SIDE_K, "k"), (sp.SIDE_V, "v")):
        s = S[name]
        params = s["params"]
        ref = np.zeros(s["total"], np.uint8)
        assert H.oracle_encode(params, side, s["X"][None], [0], ref, s["off"]) == 0
        cache = torch.zeros(s["total"], dtype=torch.uint8, device="cuda")
        pos0 = torch.zeros(1, dtype=torch.int32, device="cuda")
        st = _gpu_encode(sp, cfg, params, H.dev_params(params), side, H.to_dev(s["X"][None]), pos0, cache,
                         H.to_dev(s["off"]))
        assert st == 0
        got = cache.cpu().numpy()
        n = s["X"].shape[0]
        # every entry counts, tokens whose fp16 metadata differ included: codes within one level in at most 1e-4 of
        # the active entries, metadata within one fp16 step (a directed rounding of min/max can flip on a last-bit
        # difference of the rotation)
        tb = int(params.tile_bytes[0])
        bad, tot, dmax, mmax, n_meta = H.compare_coded_units(ref[s["off"][0]:], got[s["off"][0]:], tb, n,
                                                              params.widths[0], params.gs, side)
        assert dmax <= 1 and mmax <= 1, (dmax, mmax)
        assert bad <= MISMATCH_RATE * tot, (bad, tot)
        assert n_meta <= 2e-3 * n


@pytest.mark.parametrize("ratio,shift", [(4.0, 0), (2.0, 0), (8.0, 2)],
                         ids=["staged", "tile_larger_than_the_staging_buffer", "cache_not_16_byte_aligned"])
def test_tiny_decode_matches_oracle(sp, ratio, shift):
    """The reconstruction kernel stages packed tiles in shared memory with bulk copies when they fit and the cache
    is 16-byte aligned, and reads them in place otherwise: all three ways give the oracle's numbers."""
    wl, S = _tiny_setup(sp, ratio)
    cfg = sp.default_config()
    for side, name in ((sp.SIDE_K, "k"), (sp.SIDE_V, "v")):
        s = S[name]
        params = s["params"]
        n = 1000                                               # ragged tail
        ref = np.zeros(s["total"], np.uint8)
        H.oracle_encode(params, side, s["X"][None, :n], [0], ref, s["off"])
        yhat_ref, xhat_ref = oc.decode_unit(ref, int(params.tile_bytes[0]), n, params.w_dec[0], params.m_rot[0],
                                            params.widths[0], 64, side)
        dp = H.dev_params(params)
        for dt in (torch.float32, torch.bfloat16):
            out = torch.full((1, 1024, 128), 7.0, dtype=dt, device="cuda")
            yhat = torch.zeros((1, 1024, 128), dtype=torch.float32, device="cuda")
            cache_dev = torch.zeros(ref.size + 16, dtype=torch.uint8, device="cuda")
            cache_dev[shift:shift + ref.size] = H.to_dev(ref)
            sp.decode(cfg, side, cache_dev[shift:], H.to_dev(s["off"]), 1, 1,
                      torch.tensor([n], dtype=torch.int32, device="cuda"), n, dp["w_dec"], dp["m_rot"], dp["widths"],
                      out, yhat, 1024 * 128, 128)
            torch.cuda.synchronize()
            assert np.array_equal(yhat[0, :n].cpu().numpy(), yhat_ref)           # same fp32 operation order
            tol = TOL if dt == torch.float32 else TOL + 2.0 ** -8                  # bf16 output rounding on top
            assert H.rel_err_per_vector(out[0, :n].float().cpu().numpy(), xhat_ref) <= tol
            assert (out[0, n:] == 7.0).all()                                       # nothing written past n_tokens


def _oracle_attention(wl_group, q, n_tokens, K, V, cache_k, cache_v, mode="B"):
    pk, pv = K["params"], V["params"]
    n_units = len(n_tokens)
    idx = [u % pk.n_sets for u in range(n_units)]
    return oc.attention_units(mode, q, n_tokens, cache_k, K["off"], pk.tile_bytes[idx], cache_v, V["off"],
                              pv.tile_bytes[idx], pk.w_dec[idx], pk.m_rot[idx], pk.widths[idx], pv.w_dec[idx],
                              pv.m_rot[idx], pv.widths[idx], pk.gs, 1.0 / np.sqrt(128.0))


def _gpu_attention(sp, cfg, q_dev, batch, n_kv, n_q, seq_len, max_len, K, V, cache_k, cache_v, want_lse=True,
                   out_dtype=None, host_widths=True):
    pk, pv = K["params"], V["params"]
    dk, dv = H.dev_params(pk), H.dev_params(pv)
    out = torch.zeros((batch, n_q, 128), dtype=out_dtype or torch.float32, device="cuda")
    lse = torch.zeros((batch, n_q), dtype=torch.float32, device="cuda") if want_lse else None
    ws = torch.zeros(sp.attention_workspace_bytes(cfg, batch, n_kv, n_q, max_len), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sp.decode_attention(cfg, q_dev, batch, n_kv, n_q, H.to_dev(np.asarray(seq_len, np.int32)), max_len,
                        H.to_dev(cache_k), H.to_dev(K["off"]), H.to_dev(cache_v), H.to_dev(V["off"]), pk.n_sets,
                        dk["w_dec"], dk["m_rot"], dk["widths"], dv["w_dec"], dv["m_rot"], dv["widths"], 0.0, out, lse,
                        ws, status, pk.widths if host_widths else None, pv.widths if host_widths else None)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out.float().cpu().numpy(), None if lse is None else lse.cpu().numpy()


@pytest.mark.parametrize("host_widths", [True, False], ids=["tensor", "generic"])
@pytest.mark.parametrize("ratio", [3.0, 4.0, 5.0, 6.0, 8.0, 12.0, 16.0])
@pytest.mark.parametrize("n", [1024, 1000, 77])
def test_tiny_attention_matches_oracle(sp, ratio, n, host_widths):
    wl, S = _tiny_setup(sp, ratio)
    cfg = sp.default_config()
    caches = {}
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        s = S[name]
        c = np.zeros(s["total"], np.uint8)
        H.oracle_encode(s["params"], side, s["X"][None, :n], [0], c, s["off"])
        caches[name] = c
    q = si.draw_queries(wl, 0, 0)                                                 # [4, 128]
    ref_b, lse_b = _oracle_attention(4, q[None].astype(np.float64), [n], S["k"], S["v"], caches["k"], caches["v"])
    ref_a, _ = _oracle_attention(4, q[None].astype(np.float64), [n], S["k"], S["v"], caches["k"], caches["v"], "A")
    got, lse = _gpu_attention(sp, cfg, H.to_dev(q[None]), 1, 1, 4, [n], n, S["k"], S["v"], caches["k"], caches["v"],
                              host_widths=host_widths)
    assert H.rel_err_per_vector(got[0], ref_b[0]) <= TOL
    assert H.rel_err_per_vector(got[0], ref_a[0]) <= TOL
    assert np.abs(lse[0] - lse_b[0]).max() <= 2e-3


def test_attention_rejects_parameters_that_are_not_16_byte_aligned(sp):
    """The attention kernels read W_dec with 16-byte accesses and bulk copies: a matrix at an odd float offset is
    refused on the host (no launch), as the header says."""
    wl, S = _tiny_setup(sp, 8.0)
    cfg = sp.default_config()
    n = 256
    pk, pv = S["k"]["params"], S["v"]["params"]
    dk, dv = H.dev_params(pk), H.dev_params(pv)

    def shifted(t):                                        # the same values, one float further on
        buf = torch.zeros(t.numel() + 1, dtype=t.dtype, device="cuda")
        buf[1:] = t.reshape(-1)
        return buf[1:].view(t.shape)
    out = torch.zeros((1, 4, 128), dtype=torch.float32, device="cuda")
    ws = torch.zeros(sp.attention_workspace_bytes(cfg, 1, 1, 4, n), dtype=torch.uint8, device="cuda")
    cache = torch.zeros(int(S["k"]["total"]), dtype=torch.uint8, device="cuda")
    q = torch.zeros((1, 4, 128), dtype=torch.float32, device="cuda")
    for wk, wv in ((shifted(dk["w_dec"]), dv["w_dec"]), (dk["w_dec"], shifted(dv["w_dec"]))):
        with pytest.raises(sp.SpectraError):
            sp.decode_attention(cfg, q, 1, 1, 4, H.to_dev(np.asarray([n], np.int32)), n, cache, H.to_dev(S["k"]["off"]),
                                cache, H.to_dev(S["v"]["off"]), 1, wk, dk["m_rot"], dk["widths"], wv, dv["m_rot"],
                                dv["widths"], 0.0, out, None, ws, None, pk.widths, pv.widths)
    torch.cuda.synchronize()


def _multi_unit_setup(wl, n_seq, n_tokens, ratio, gs=64, seq_lens=None):
    """One layer of a (possibly GQA-7) workload: per-head parameter sets shared by the sequences of the batch."""
    S = {}
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        X = H.draw_units(wl, 0, side, n_seq, n_tokens)                           # [n_seq*H, n, d]
        params = H.fit_params([X[h][:min(n_tokens, wl.n_fit)] for h in range(wl.kv_heads)], ratio, gs=gs)
        n_units = n_seq * wl.kv_heads
        off, total = H.cache_layout(params, n_units, n_tokens)
        cache = np.zeros(total, np.uint8)
        lens = seq_lens if seq_lens is not None else [n_tokens] * n_seq
        for u in range(n_units):
            nn = lens[u // wl.kv_heads]
            if nn:
                H.oracle_encode(H.Params(params.w_enc[[u % wl.kv_heads]], params.w_dec[[u % wl.kv_heads]],
                                         params.m_rot[[u % wl.kv_heads]], params.widths[[u % wl.kv_heads]], gs),
                                side, X[u][None, :nn], [0], cache[off[u]:], np.zeros(1, np.int64))
        S[name] = dict(params=params, off=off, total=total, cache=cache)
    return S


@pytest.mark.parametrize("name,ratio,gs", [("llama", 8.0, 64), ("qwen", 12.0, 64), ("llama", 4.0, 32),
                                           ("llama", 8.0, 128)])
def test_batched_gqa_attention_matches_oracle(sp, name, ratio, gs):
    base = si.WORKLOADS["llama1" if name == "llama" else "qwen28"]
    wl = dataclasses.replace(base, kv_heads=2, q_heads=2 * base.group, n_fit=512)
    n_seq, n_tokens = 3, 700
    seq_lens = [700, 0, 333]                                                      # full, empty, ragged
    S = _multi_unit_setup(wl, n_seq, n_tokens, ratio, gs, seq_lens)
    cfg = sp.default_config(scale_group=gs)
    q = np.stack([si.draw_queries(wl, 0, s) for s in range(n_seq)])               # [n_seq, Hq, d]
    G = wl.group
    n_units = n_seq * wl.kv_heads
    q_units = q.reshape(n_seq, wl.kv_heads, G, 128).reshape(n_units, G, 128).astype(np.float64)
    unit_lens = [seq_lens[u // wl.kv_heads] for u in range(n_units)]
    live = [u for u in range(n_units) if unit_lens[u] > 0]
    K, V = S["k"], S["v"]
    got, lse = _gpu_attention(sp, cfg, H.to_dev(q), n_seq, wl.kv_heads, wl.q_heads, seq_lens, n_tokens, K, V,
                              K["cache"], V["cache"])
    got_units = got.reshape(n_seq, wl.kv_heads, G, 128).reshape(n_units, G, 128)
    lse_units = lse.reshape(n_seq, wl.kv_heads, G).reshape(n_units, G)
    for u in range(n_units):
        p = u % wl.kv_heads
        if unit_lens[u] == 0:
            assert (got_units[u] == 0).all() and np.isneginf(lse_units[u]).all()
            continue
        ref, lref = oc.attention_units("B", q_units[u][None], [unit_lens[u]], K["cache"], [K["off"][u]],
                                       [K["params"].tile_bytes[p]], V["cache"], [V["off"][u]],
                                       [V["params"].tile_bytes[p]], K["params"].w_dec[[p]], K["params"].m_rot[[p]],
                                       K["params"].widths[[p]], V["params"].w_dec[[p]], V["params"].m_rot[[p]],
                                       V["params"].widths[[p]], gs, 1.0 / np.sqrt(128.0))
        assert H.rel_err_per_vector(got_units[u], ref[0]) <= TOL, u
        assert np.abs(lse_units[u] - lref[0]).max() <= 2e-3
    assert live


def test_attention_bf16_query_and_output(sp):
    wl, S = _tiny_setup(sp, 8.0)
    cfg = sp.default_config()
    n = 512
    caches = {}
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        s = S[name]
        c = np.zeros(s["total"], np.uint8)
        H.oracle_encode(s["params"], side, s["X"][None, :n], [0], c, s["off"])
        caches[name] = c
    q = si.to_bf16_f32(si.draw_queries(wl, 0, 0))
    ref, _ = _oracle_attention(4, q[None].astype(np.float64), [n], S["k"], S["v"], caches["k"], caches["v"])
    got, _ = _gpu_attention(sp, cfg, H.to_dev(q[None]).to(torch.bfloat16), 1, 1, 4, [n], n, S["k"], S["v"],
                            caches["k"], caches["v"], want_lse=False, out_dtype=torch.bfloat16)
    assert H.rel_err_per_vector(got[0], ref[0]) <= TOL + 2.0 ** -8


# ----------------------------------------------------------------------------- basis fit

@pytest.mark.parametrize("gain_mode", [ofit.GAIN_ROTATE, ofit.GAIN_SQRT, ofit.GAIN_WHITEN])
def test_fit_basis_invariants_and_spectrum(sp, gain_mode):
    wl = si.WORKLOADS["tiny"]
    n_units, n = 3, 1024
    X = np.stack([si.draw_unit(wl, 0, h, si.SIDE_K if h < 2 else si.SIDE_V, 0, n_tokens=n) for h in range(n_units)])
    X[1] += 0.5                                                                    # a unit with a clear mean
    cfg = sp.default_config(gain_mode=gain_mode)
    xd = H.to_dev(X)
    f32 = dict(dtype=torch.float32, device="cuda")
    w_enc, w_dec, U = (torch.zeros((n_units, 128, 128), **f32) for _ in range(3))
    m_rot, var, lam = (torch.zeros((n_units, 128), **f32) for _ in range(3))
    ws = torch.zeros(sp.fit_workspace_bytes(cfg, n_units), dtype=torch.uint8, device="cuda")
    sp.fit_basis(cfg, xd, n_units, n, n * 128, 128, w_enc, w_dec, m_rot, var, lam, U, ws)
    torch.cuda.synchronize()
    for u in range(n_units):
        ref = ofit.fit_basis(X[u].astype(np.float64), gain_mode)
        Ug = U[u].cpu().numpy().astype(np.float64)
        assert np.abs(Ug.T @ Ug - np.eye(128)).max() <= 5e-6                       # fp32 storage of an fp64 basis
        lam_g = lam[u].cpu().numpy().astype(np.float64)
        assert np.abs(lam_g - ref["lam"]).max() <= 2e-6 * ref["lam"][0]
        off = Ug.T @ ref["C"] @ Ug
        assert np.abs(off - np.diag(np.diag(off))).max() <= 5e-6 * ref["lam"][0]
        assert (Ug[np.argmax(np.abs(Ug), axis=0), np.arange(128)] > 0).all()
        we, wd = w_enc[u].cpu().numpy().astype(np.float64), w_dec[u].cpu().numpy().astype(np.float64)
        assert np.abs(we @ wd - np.eye(128)).max() <= 2e-5
        # rotated statistics, measured directly on the data with the GPU's own transform
        Y = X[u].astype(np.float64) @ we
        assert np.allclose(Y.mean(axis=0), m_rot[u].cpu().numpy(), rtol=2e-4, atol=2e-5 * np.abs(Y).max())
        v_meas = Y.var(axis=0)
        v_gpu = var[u].cpu().numpy().astype(np.float64)
        if gain_mode == ofit.GAIN_WHITEN:
            assert np.allclose(v_meas, 1.0, rtol=2e-3)
            assert np.allclose(v_gpu, ref["v_alloc"], rtol=2e-3, atol=1e-7 * ref["lam"][0])
        else:
            assert np.allclose(v_gpu, v_meas, rtol=2e-3, atol=1e-6 * v_meas.max())
        # the fitted basis allocates like the oracle's basis does
        widths = torch.zeros((1, 128), dtype=torch.uint8, device="cuda")
        sp.alloc_bits(cfg, var[u:u + 1].contiguous(), 1, 8.0, widths)
        wg = widths.cpu().numpy()[0].astype(np.int64)
        wr = ofit.alloc_bits(ref["v_alloc"].astype(np.float32), 256).astype(np.int64)
        assert wg.sum() == 256 and np.abs(wg - wr).max() <= 1 and (wg != wr).mean() <= 0.1


def test_fit_basis_bf16_strided_input(sp):
    """The fit reads a [batch, heads, tokens, d] bf16 cache in place: sequence 0, first n_fit tokens of each head."""
    wl = si.WORKLOADS["llama1"]
    heads, n_all, n_fit = 2, 640, 512
    X = np.stack([si.draw_unit(wl, 0, h, si.SIDE_K, 0, n_tokens=n_all) for h in range(heads)])
    cfg = sp.default_config()
    xd = H.to_dev(X).to(torch.bfloat16)
    f32 = dict(dtype=torch.float32, device="cuda")
    w_enc, w_dec = (torch.zeros((heads, 128, 128), **f32) for _ in range(2))
    m_rot, var, lam = (torch.zeros((heads, 128), **f32) for _ in range(3))
    ws = torch.zeros(sp.fit_workspace_bytes(cfg, heads), dtype=torch.uint8, device="cuda")
    sp.fit_basis(cfg, xd, heads, n_fit, n_all * 128, 128, w_enc, w_dec, m_rot, var, lam, None, ws)
    torch.cuda.synchronize()
    for h in range(heads):
        ref = ofit.fit_basis(X[h, :n_fit].astype(np.float64), ofit.GAIN_SQRT)
        assert np.abs(lam[h].cpu().numpy() - ref["lam"]).max() <= 2e-6 * ref["lam"][0]


# ----------------------------------------------------------------------------- whole pipeline on the GPU, config 0

def test_tiny_whole_pipeline_on_gpu_agrees_with_whole_oracle(sp):
    """Fit, allocate, encode and attend entirely on the GPU; the oracle does the same from the same raw data.
    The two bases may differ inside near-degenerate eigen-subspaces, so the comparison is on what is unique:
    the attention output against the oracle's own coded result and against dense attention."""
    wl = si.WORKLOADS["tiny"]
    cfg = sp.default_config()
    n = wl.n_tokens
    f32 = dict(dtype=torch.float32, device="cuda")
    dev = {}
    Xs = {}
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        X = si.draw_unit(wl, 0, 0, side, 0)
        Xs[name] = X
        xd = H.to_dev(X[None])
        w_enc, w_dec = (torch.zeros((1, 128, 128), **f32) for _ in range(2))
        m_rot, var = (torch.zeros((1, 128), **f32) for _ in range(2))
        ws = torch.zeros(sp.fit_workspace_bytes(cfg, 1), dtype=torch.uint8, device="cuda")
        sp.fit_basis(cfg, xd, 1, n, n * 128, 128, w_enc, w_dec, m_rot, var, None, None, ws)
        widths = torch.zeros((1, 128), dtype=torch.uint8, device="cuda")
        sp.alloc_bits(cfg, var, 1, wl.ratio, widths)
        tb = sp.tile_bytes(cfg, widths.cpu().numpy()[0])
        cache = torch.zeros(tb * (n // 128), dtype=torch.uint8, device="cuda")
        off = torch.zeros(1, dtype=torch.int64, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        sp.encode(cfg, side, xd, 0, 1, 1, torch.zeros(1, dtype=torch.int32, device="cuda"), n, n * 128, 128, w_enc,
                  m_rot, widths, cache, off, status)
        assert _sync_status(status) == 0
        dev[name] = dict(w_dec=w_dec, m_rot=m_rot, widths=widths, cache=cache, off=off)
        assert 16 * int(widths.sum().item()) == 16 * 512
    q = si.draw_queries(wl, 0, 0)
    out = torch.zeros((1, 4, 128), **f32)
    ws = torch.zeros(sp.attention_workspace_bytes(cfg, 1, 1, 4, n), dtype=torch.uint8, device="cuda")
    k, v = dev["k"], dev["v"]
    sp.decode_attention(cfg, H.to_dev(q[None]), 1, 1, 4, torch.tensor([n], dtype=torch.int32, device="cuda"), n,
                        k["cache"], k["off"], v["cache"], v["off"], 1, k["w_dec"], k["m_rot"], k["widths"],
                        v["w_dec"], v["m_rot"], v["widths"], 0.0, out, None, ws, None)
    torch.cuda.synchronize()
    got = out.cpu().numpy()[0]
    # the oracle's whole pipeline
    S = {}
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        params = H.fit_params([Xs[name]], wl.ratio)
        off, total = H.cache_layout(params, 1, n)
        c = np.zeros(total, np.uint8)
        H.oracle_encode(params, side, Xs[name][None], [0], c, off)
        S[name] = dict(params=params, off=off, cache=c)
    ref, _ = _oracle_attention(4, q[None].astype(np.float64), [n], S["k"], S["v"], S["k"]["cache"], S["v"]["cache"])
    s = q.astype(np.float64) @ Xs["k"].astype(np.float64).T / np.sqrt(128.0)
    p = np.exp(s - s.max(axis=1, keepdims=True))
    dense = (p / p.sum(axis=1, keepdims=True)) @ Xs["v"].astype(np.float64)
    err_gpu = np.linalg.norm(got - dense) / np.linalg.norm(dense)
    err_ref = np.linalg.norm(ref[0] - dense) / np.linalg.norm(dense)
    assert err_gpu <= 1.5 * err_ref + 1e-3                     # same quality as the oracle's codec at 4x
    assert H.rel_err_per_vector(got, ref[0]) <= 0.05           # and close to it (bases differ in degenerate tails)


@pytest.mark.parametrize("name,tensor_path", [("tiny", True), ("tiny", False)])
def test_fused_decode_step_equals_separate_calls(sp, name, tensor_path):
    """spectra_decode_step = spectra_encode (K), spectra_encode (V), spectra_decode_attention: same cache bytes, same
    outputs (the separate calls are the ones the other tests compare with the oracle)."""
    import dataclasses
    from paper_2608_07915_b200 import harness
    wl = dataclasses.replace(si.WORKLOADS[name], batch=2)
    models = []
    for fused in (True, False):
        m = harness.CodedModelCache(wl, layers=1, batch=2, extra_tokens=256)
        m.tensor_path = tensor_path
        m.build()
        models.append(m)
    gen = torch.Generator(device="cuda").manual_seed(5)
    outs = []
    dt = torch.float32 if wl.dtype == "f32" else torch.bfloat16
    steps = [(torch.randn((1, 2, wl.q_heads, 128), generator=gen, device="cuda").to(dt),
              torch.randn((1, 2 * wl.kv_heads, 128), generator=gen, device="cuda").to(dt),
              torch.randn((1, 2 * wl.kv_heads, 128), generator=gen, device="cuda").to(dt)) for _ in range(130)]
    for m, fused in zip(models, (True, False)):
        out = torch.zeros((1, 2, wl.q_heads, 128), dtype=torch.float32, device="cuda")
        for q, nk, nv in steps:                      # crosses a tile boundary (130 appended tokens)
            m.decode_step(q, nk, nv, out, fused=fused)
        torch.cuda.synchronize()
        assert int(m.status.item()) == 0
        outs.append(out.clone())
    for side in (0, 1):
        assert torch.equal(models[0].side[0][side].cache, models[1].side[0][side].cache)
    if tensor_path:
        assert torch.equal(outs[0], outs[1])
    else:   # the CUDA-core kernel sums with shared-memory float atomics: equal up to summation order
        assert torch.allclose(outs[0], outs[1], rtol=1e-5, atol=1e-6)


def test_fused_decode_step_skips_empty_sequences(sp):
    """A sequence of length 0 in a fused step gets no append (its cache stays as it was) and a zero output row."""
    import dataclasses
    from paper_2608_07915_b200 import harness
    wl = dataclasses.replace(si.WORKLOADS["tiny"], batch=2)
    m = harness.CodedModelCache(wl, layers=1, batch=2, extra_tokens=128)
    m.build()
    before = [m.side[0][s].cache.clone() for s in (0, 1)]
    gen = torch.Generator(device="cuda").manual_seed(6)
    q = torch.randn((2, wl.q_heads, 128), generator=gen, device="cuda")
    nk = torch.randn((2 * wl.kv_heads, 128), generator=gen, device="cuda")
    nv = torch.randn((2 * wl.kv_heads, 128), generator=gen, device="cuda")
    out = torch.full((2, wl.q_heads, 128), 3.0, dtype=torch.float32, device="cuda")
    m.seq_len += 1
    m.seq_len[1] = 0
    m.step_layer(0, q, nk, nv, out)
    torch.cuda.synchronize()
    assert int(m.status.item()) == 0
    assert (out[1] == 0).all() and torch.isfinite(out[0]).all() and (out[0] != 3.0).any()
    for s in (0, 1):
        ls = m.side[0][s]
        for u in range(wl.kv_heads, 2 * wl.kv_heads):            # units of the empty sequence
            a = int(ls.unit_offset_host[u])
            e = int(ls.unit_offset_host[u + 1]) if u + 1 < 2 * wl.kv_heads else ls.cache.numel()
            assert torch.equal(ls.cache[a:e], before[s][a:e])
        assert not torch.equal(ls.cache, before[s])               # the other sequence did get its token


@pytest.mark.parametrize("tensor_path", [True, False], ids=["tensor", "generic"])
def test_inputs_with_a_large_mean_reconstruction_attention_and_fused_step(sp, tensor_path):
    """The synthetic recipe is zero-mean, which leaves the rotated means m' (removed before quantisation, Sec. 3.1;
    restored by the reconstruction, and in the latent-space attention through q'.m'_K in lse and + m'_V before the
    lift) at sampling-noise size.  Here every vector is shifted by one standard deviation per channel, so that m'
    is as large as the data: reconstruction, attention and the fused decode step against the oracle."""
    wl = si.WORKLOADS["tiny"]
    cfg = sp.default_config()
    n, ratio = 600, 8.0
    S, caches = {}, {}
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        X = si.draw_unit(wl, 0, 0, side, 0, n_tokens=n + 1) + si.mean_offset(wl, 0, 0, side)[None]
        params = H.fit_params([X[:n]], ratio)
        assert np.abs(params.m_rot[0]).max() > 0.5 * np.abs((X[:n] @ params.w_enc[0]).std(axis=0)).max()
        off, total = H.cache_layout(params, 1, n + 128)
        c = np.zeros(total, np.uint8)
        assert H.oracle_encode(params, side, X[None, :n], [0], c, off) == 0
        S[name] = dict(X=X, params=params, off=off, total=total)
        caches[name] = c
        # reconstruction of the oracle's bytes
        yhat_ref, xhat_ref = oc.decode_unit(c, int(params.tile_bytes[0]), n, params.w_dec[0], params.m_rot[0],
                                            params.widths[0], 64, side)
        dp = H.dev_params(params)
        out = torch.zeros((1, n, 128), dtype=torch.float32, device="cuda")
        yhat = torch.zeros((1, n, 128), dtype=torch.float32, device="cuda")
        sp.decode(cfg, side, H.to_dev(c), H.to_dev(off), 1, 1, torch.tensor([n], dtype=torch.int32, device="cuda"), n,
                  dp["w_dec"], dp["m_rot"], dp["widths"], out, yhat, n * 128, 128)
        torch.cuda.synchronize()
        assert np.array_equal(yhat[0].cpu().numpy(), yhat_ref)
        assert H.rel_err_per_vector(out[0].cpu().numpy(), xhat_ref) <= TOL
    q = si.draw_queries(wl, 0, 0)
    hw = tensor_path
    ref_b, lse_b = _oracle_attention(4, q[None].astype(np.float64), [n], S["k"], S["v"], caches["k"], caches["v"])
    ref_a, lse_a = _oracle_attention(4, q[None].astype(np.float64), [n], S["k"], S["v"], caches["k"], caches["v"], "A")
    got, lse = _gpu_attention(sp, cfg, H.to_dev(q[None]), 1, 1, 4, [n], n + 128, S["k"], S["v"], caches["k"],
                              caches["v"], host_widths=hw)
    assert H.rel_err_per_vector(got[0], ref_b[0]) <= TOL and H.rel_err_per_vector(got[0], ref_a[0]) <= TOL
    assert np.abs(lse[0] - lse_b[0]).max() <= 2e-3 and np.abs(lse[0] - lse_a[0]).max() <= 2e-3
    # the fused step: appends token n of both sides, then attends over n + 1 tokens
    pk, pv = S["k"]["params"], S["v"]["params"]
    dk, dv = H.dev_params(pk), H.dev_params(pv)
    ck, cv = H.to_dev(caches["k"]), H.to_dev(caches["v"])
    out = torch.zeros((1, 4, 128), dtype=torch.float32, device="cuda")
    lse_d = torch.zeros((1, 4), dtype=torch.float32, device="cuda")
    ws = torch.zeros(sp.attention_workspace_bytes(cfg, 1, 1, 4, n + 128), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    q2 = si.draw_queries(wl, 0, 0, step=1)
    sp.decode_step(cfg, H.to_dev(q2[None]), H.to_dev(S["k"]["X"][n][None]), H.to_dev(S["v"]["X"][n][None]), 1, 1, 4,
                   torch.tensor([n + 1], dtype=torch.int32, device="cuda"), n + 128, ck, H.to_dev(S["k"]["off"]), cv,
                   H.to_dev(S["v"]["off"]), 1, dk["w_enc"], dk["w_dec"], dk["m_rot"], dk["widths"], dv["w_enc"],
                   dv["w_dec"], dv["m_rot"], dv["widths"], 0.0, out, lse_d, ws, status, pk.widths if hw else None,
                   pv.widths if hw else None)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    held = {"k": ck.cpu().numpy(), "v": cv.cpu().numpy()}
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        pr = S[name]["params"]
        ref = caches[name].copy()
        assert H.oracle_encode(pr, side, S[name]["X"][None, n:n + 1], [n], ref, S[name]["off"]) == 0
        bad, tot, dmax, mmax, _ = H.compare_coded_units(ref, held[name], int(pr.tile_bytes[0]), n + 1, pr.widths[0], 64,
                                                        side)
        assert dmax <= 1 and mmax <= 1 and bad <= 2
    ref2, lse2 = _oracle_attention(4, q2[None].astype(np.float64), [n + 1], S["k"], S["v"], held["k"], held["v"])
    assert H.rel_err_per_vector(out.cpu().numpy()[0], ref2[0]) <= TOL
    assert np.abs(lse_d.cpu().numpy()[0] - lse2[0]).max() <= 2e-3


def test_appends_beyond_the_capacity_are_reported_not_written(sp):
    """spectra_encode with a capacity: tokens at positions >= capacity_tokens are not written and the status word gets
    SPECTRA_STATUS_CAPACITY, on the append kernel (a few tokens), the CUDA-core bulk kernel (fp32) and the
    tensor-core bulk kernel (bf16).  The buffer is followed by a guard region that must stay untouched."""
    wl = si.WORKLOADS["tiny"]
    cfg = sp.default_config()
    X = si.draw_unit(wl, 0, 0, si.SIDE_K, 0, n_tokens=512)
    params = H.fit_params([X], 8.0)
    dp = H.dev_params(params)
    tb = int(params.tile_bytes[0])
    cap = 256                                              # two tiles
    assert sp.cache_bytes(cfg, params.widths[0], cap) == 2 * tb
    for dt, first, n_new in ((torch.float32, 250, 10), (torch.float32, 100, 300), (torch.bfloat16, 100, 300),
                             (torch.float32, 256, 4)):
        ref = np.zeros(2 * tb, np.uint8)
        n_fit = max(0, min(cap - first, n_new))
        xs = si.to_bf16_f32(X[first:first + n_new]) if dt == torch.bfloat16 else X[first:first + n_new]
        if n_fit:
            assert H.oracle_encode(params, si.SIDE_K, xs[None, :n_fit], [first], ref, np.zeros(1, np.int64)) == 0
        buf = torch.full((2 * tb + 4096,), 0x5C, dtype=torch.uint8, device="cuda")
        buf[:2 * tb] = 0
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        sp.encode(cfg, si.SIDE_K, H.to_dev(xs[None]).to(dt), 0, 1, 1, torch.tensor([first], dtype=torch.int32, device="cuda"),
                  n_new, n_new * 128, 128, dp["w_enc"], dp["m_rot"], dp["widths"], buf,
                  torch.zeros(1, dtype=torch.int64, device="cuda"), status, capacity_tokens=cap)
        torch.cuda.synchronize()
        assert int(status.item()) == sp.STATUS_CAPACITY
        got = buf.cpu().numpy()
        assert (got[2 * tb:] == 0x5C).all()                # nothing past the buffer
        if n_fit:
            bad, tot, dmax, mmax, _ = H.compare_coded_units(ref, got[:2 * tb], tb, cap, params.widths[0], 64, si.SIDE_K)
            assert dmax <= 1 and mmax <= 1 and bad <= 3
        else:
            assert not got[:2 * tb].any()
    # within the capacity: no bit
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    buf = torch.zeros(2 * tb, dtype=torch.uint8, device="cuda")
    sp.encode(cfg, si.SIDE_K, H.to_dev(X[None, :256]), 0, 1, 1, torch.zeros(1, dtype=torch.int32, device="cuda"), 256,
              256 * 128, 128, dp["w_enc"], dp["m_rot"], dp["widths"], buf, torch.zeros(1, dtype=torch.int64, device="cuda"),
              status, capacity_tokens=cap)
    torch.cuda.synchronize()
    assert int(status.item()) == 0


@pytest.mark.parametrize("tensor_path", [True, False], ids=["tensor", "generic"])
def test_sequence_longer_than_max_seq_len_is_reported_and_skipped(sp, tensor_path):
    """Attention and the fused step treat max_seq_len as the capacity: a sequence whose seq_len exceeds it sets
    SPECTRA_STATUS_CAPACITY, gets no append and a zero output row; the other sequence is unaffected."""
    import dataclasses
    from paper_2608_07915_b200 import harness
    wl = dataclasses.replace(si.WORKLOADS["tiny"], batch=2)
    m = harness.CodedModelCache(wl, layers=1, batch=2, extra_tokens=128)
    m.tensor_path = tensor_path
    m.build()
    before = [m.side[0][s].cache.clone() for s in (0, 1)]
    gen = torch.Generator(device="cuda").manual_seed(8)
    q = torch.randn((2, wl.q_heads, 128), generator=gen, device="cuda")
    nk = torch.randn((2 * wl.kv_heads, 128), generator=gen, device="cuda")
    nv = torch.randn((2 * wl.kv_heads, 128), generator=gen, device="cuda")
    ref = torch.zeros((2, wl.q_heads, 128), dtype=torch.float32, device="cuda")
    m.seq_len += 1
    m.step_layer(0, q, nk, nv, ref)                       # both sequences in range
    torch.cuda.synchronize()
    assert int(m.status.item()) == 0
    for s in (0, 1):
        m.side[0][s].cache.copy_(before[s])
    m.seq_len[1] = m.cap_tokens + 1                        # beyond what the buffers hold
    out = torch.full((2, wl.q_heads, 128), 3.0, dtype=torch.float32, device="cuda")
    m.step_layer(0, q, nk, nv, out)
    torch.cuda.synchronize()
    assert int(m.status.item()) == sp.STATUS_CAPACITY
    assert (out[1] == 0).all()
    if tensor_path:
        assert torch.equal(out[0], ref[0])
    else:
        assert torch.allclose(out[0], ref[0], rtol=1e-5, atol=1e-6)
    for s in (0, 1):
        ls = m.side[0][s]
        a = int(ls.unit_offset_host[wl.kv_heads])
        assert torch.equal(ls.cache[a:], before[s][a:])   # the units of the out-of-range sequence were not touched


def test_tensor_core_path_refuses_units_whose_widths_differ_from_the_host_copy(sp):
    """The host sizes the shared-memory tile slots from its copy of the widths.  If the widths on the device ask for
    larger tiles (a caller's mistake), the kernels must not copy them: the unit is skipped, SPECTRA_STATUS_BAD_LAYOUT
    is set, and the call completes with finite outputs."""
    wl, S = _tiny_setup(sp, 4.0)
    cfg = sp.default_config()
    n = 512
    caches = {}
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        c = np.zeros(S[name]["total"], np.uint8)
        H.oracle_encode(S[name]["params"], side, S[name]["X"][None, :n], [0], c, S[name]["off"])
        caches[name] = c
    pk, pv = S["k"]["params"], S["v"]["params"]
    dk, dv = H.dev_params(pk), H.dev_params(pv)
    host_k = np.minimum(pk.widths, 2).astype(np.uint8)      # the host believes in narrower channels: smaller tiles
    host_v = np.minimum(pv.widths, 2).astype(np.uint8)
    assert sp.attention_path(cfg, 1, 4, 1, host_k, host_v) == sp.PATH_TENSOR_CORE
    q = H.to_dev(si.draw_queries(wl, 0, 0)[None])
    out = torch.full((1, 4, 128), 3.0, dtype=torch.float32, device="cuda")
    ws = torch.zeros(sp.attention_workspace_bytes(cfg, 1, 1, 4, n), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sp.decode_attention(cfg, q, 1, 1, 4, H.to_dev(np.asarray([n], np.int32)), n, H.to_dev(caches["k"]),
                        H.to_dev(S["k"]["off"]), H.to_dev(caches["v"]), H.to_dev(S["v"]["off"]), 1, dk["w_dec"],
                        dk["m_rot"], dk["widths"], dv["w_dec"], dv["m_rot"], dv["widths"], 0.0, out, None, ws, status,
                        host_k, host_v)
    torch.cuda.synchronize()
    assert int(status.item()) == sp.STATUS_BAD_LAYOUT
    assert torch.isfinite(out).all()


def test_attention_with_value_outlier_tokens_that_carry_the_probability_mass(sp):
    """A few late tokens whose value vectors are 30 times larger than the rest, one of them with the dominant score:
    probability times value range is then far above what the first tiles suggested.  The kernel must follow
    (its fp16 operand of the value contraction is rescaled when a tile needs more headroom), not saturate."""
    wl = si.WORKLOADS["tiny"]
    cfg = sp.default_config()
    n = 900
    q = si.draw_queries(wl, 0, 0)
    S, caches = {}, {}
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        X = si.draw_unit(wl, 0, 0, side, 0, n_tokens=n).copy()
        if side == si.SIDE_V:
            X[700:705] *= 30.0
        else:
            X[702] = 2.0 * q[0]                                  # head 0 attends to token 702 almost exclusively
        params = H.fit_params([X[:512]], 8.0)
        off, total = H.cache_layout(params, 1, n)
        c = np.zeros(total, np.uint8)
        assert H.oracle_encode(params, side, X[None], [0], c, off) == 0
        S[name] = dict(X=X, params=params, off=off, total=total)
        caches[name] = c
    ref_b, lse_b = _oracle_attention(4, q[None].astype(np.float64), [n], S["k"], S["v"], caches["k"], caches["v"])
    ref_a, _ = _oracle_attention(4, q[None].astype(np.float64), [n], S["k"], S["v"], caches["k"], caches["v"], "A")
    got, lse = _gpu_attention(sp, cfg, H.to_dev(q[None]), 1, 1, 4, [n], n, S["k"], S["v"], caches["k"], caches["v"])
    assert np.abs(ref_b[0, 0]).max() > 5 * np.abs(ref_b[0, 1:]).max()     # head 0 did land on an outlier token
    assert H.rel_err_per_vector(got[0], ref_b[0]) <= TOL and H.rel_err_per_vector(got[0], ref_a[0]) <= TOL
    assert np.abs(lse[0] - lse_b[0]).max() <= 2e-3


@pytest.mark.parametrize("dt", ["f32", "bf16"])
def test_paged_caches_give_the_same_bytes_and_outputs_as_contiguous_ones(sp, dt):
    """Paged caches (a page table over tile-sized pages of a pool shared by the sequences of a head): bulk encode,
    appends, reconstruction, attention on both kernels and the fused step must produce, page by page, the bytes of
    the contiguous layout, and the same outputs; the attention is also compared with the oracle on the gathered
    bytes."""
    wl = si.WORKLOADS["tiny"]
    cfg = sp.default_config()
    tdt = torch.float32 if dt == "f32" else torch.bfloat16
    n_seq, n0, cap = 2, 600, 768                       # 600 cached tokens (4 full tiles + 88), room for 6 tiles
    n_tiles = cap // 128
    rng = np.random.default_rng(17)
    perm = rng.permutation(2 * n_tiles + 3)            # pool of 15 pages, 12 used, interleaved between the sequences
    table = np.stack([perm[:n_tiles], perm[n_tiles:2 * n_tiles]]).astype(np.int32)
    tab_dev = H.to_dev(table)
    zero_off = torch.zeros(n_seq, dtype=torch.int64, device="cuda")     # both sequences share the head's pool
    S = {}
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        X = np.stack([si.draw_unit(wl, 0, 0, side, s, n_tokens=n0 + 2) for s in range(n_seq)])
        if dt == "bf16":
            X = si.to_bf16_f32(X)
        params = H.fit_params([X[0, :512]], 8.0)
        tb = int(params.tile_bytes[0])
        off_c = np.array([0, n_tiles * tb], np.int64)
        S[name] = dict(X=X, params=params, tb=tb, off=off_c, dp=H.dev_params(params),
                       cont=torch.zeros(2 * n_tiles * tb, dtype=torch.uint8, device="cuda"),
                       pool=torch.full((len(perm) * tb,), 0xEE, dtype=torch.uint8, device="cuda"))

    def gathered(name):
        c = S[name]
        pool = c["pool"].cpu().numpy().reshape(len(perm), c["tb"])
        return np.concatenate([pool[table[s, t]] for s in range(n_seq) for t in range(n_tiles)])

    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    pos = torch.zeros(n_seq, dtype=torch.int32, device="cuda")
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        c = S[name]
        x = H.to_dev(c["X"][:, :n0]).to(tdt)
        for cache, off, kw in ((c["cont"], H.to_dev(c["off"]), {}),
                               (c["pool"], zero_off, dict(tile_table=tab_dev, table_stride=n_tiles))):
            sp.encode(cfg, side, x, 0, n_seq, 1, pos, n0, x.stride(0), 128, c["dp"]["w_enc"], c["dp"]["m_rot"],
                      c["dp"]["widths"], cache, off, status, capacity_tokens=cap, **kw)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for name in ("k", "v"):
        c = S[name]
        g = gathered(name).reshape(n_seq, n_tiles, c["tb"])
        r = c["cont"].cpu().numpy().reshape(n_seq, n_tiles, c["tb"])
        assert np.array_equal(g[:, :5], r[:, :5])                       # the five tiles that hold tokens
        pool = c["pool"].cpu().numpy().reshape(len(perm), c["tb"])
        for pg in perm[2 * n_tiles:]:
            assert (pool[pg] == 0xEE).all()                              # pages outside the tables stay untouched
    # reconstruction
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        c = S[name]
        outs = []
        for cache, off, kw in ((c["cont"], H.to_dev(c["off"]), {}),
                               (c["pool"], zero_off, dict(tile_table=tab_dev, table_stride=n_tiles))):
            o = torch.zeros((n_seq, n0, 128), dtype=torch.float32, device="cuda")
            y = torch.zeros((n_seq, n0, 128), dtype=torch.float32, device="cuda")
            sp.decode(cfg, side, cache, off, n_seq, 1, torch.full((n_seq,), n0, dtype=torch.int32, device="cuda"), n0,
                      c["dp"]["w_dec"], c["dp"]["m_rot"], c["dp"]["widths"], o, y, n0 * 128, 128, status, **kw)
            torch.cuda.synchronize()
            outs.append((o, y))
        assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    # attention on both kernels, then two fused steps (the second crosses nothing; the tail tile grows in place)
    k, v = S["k"], S["v"]
    q = H.to_dev(np.stack([si.draw_queries(wl, 0, s) for s in range(n_seq)]))
    ws = torch.zeros(sp.attention_workspace_bytes(cfg, n_seq, 1, 4, cap), dtype=torch.uint8, device="cuda")
    seq = torch.full((n_seq,), n0, dtype=torch.int32, device="cuda")
    for hw in (True, False):
        res = []
        for paged in (False, True):
            o = torch.zeros((n_seq, 4, 128), dtype=torch.float32, device="cuda")
            l = torch.zeros((n_seq, 4), dtype=torch.float32, device="cuda")
            kw = dict(tile_table_k=tab_dev, tile_table_v=tab_dev, table_stride=n_tiles) if paged else {}
            sp.decode_attention(cfg, q, n_seq, 1, 4, seq, cap, k["pool"] if paged else k["cont"],
                                zero_off if paged else H.to_dev(k["off"]), v["pool"] if paged else v["cont"],
                                zero_off if paged else H.to_dev(v["off"]), 1, k["dp"]["w_dec"], k["dp"]["m_rot"],
                                k["dp"]["widths"], v["dp"]["w_dec"], v["dp"]["m_rot"], v["dp"]["widths"], 0.0, o, l, ws,
                                status, k["params"].widths if hw else None, v["params"].widths if hw else None, **kw)
            torch.cuda.synchronize()
            res.append((o.cpu().numpy(), l.cpu().numpy()))
        if hw:
            assert np.array_equal(res[0][0], res[1][0]) and np.array_equal(res[0][1], res[1][1])
        else:
            assert np.allclose(res[0][0], res[1][0], rtol=1e-5, atol=1e-6)
        gk, gv = gathered("k"), gathered("v")
        ref, lse = oc.attention_units("B", q.cpu().numpy().astype(np.float64).reshape(n_seq, 4, 128), [n0] * n_seq, gk,
                                      k["off"], [k["tb"]] * n_seq, gv, v["off"], [v["tb"]] * n_seq,
                                      np.repeat(k["params"].w_dec, n_seq, 0), np.repeat(k["params"].m_rot, n_seq, 0),
                                      np.repeat(k["params"].widths, n_seq, 0), np.repeat(v["params"].w_dec, n_seq, 0),
                                      np.repeat(v["params"].m_rot, n_seq, 0), np.repeat(v["params"].widths, n_seq, 0),
                                      64, 1.0 / np.sqrt(128.0))
        assert H.rel_err_per_vector(res[1][0], ref) <= TOL
    for step in range(2):
        seq += 1
        nk = H.to_dev(k["X"][:, n0 + step]).to(tdt).contiguous()
        nv = H.to_dev(v["X"][:, n0 + step]).to(tdt).contiguous()
        res = []
        for paged in (False, True):
            o = torch.zeros((n_seq, 4, 128), dtype=torch.float32, device="cuda")
            kw = dict(tile_table_k=tab_dev, tile_table_v=tab_dev, table_stride=n_tiles) if paged else {}
            sp.decode_step(cfg, q, nk, nv, n_seq, 1, 4, seq, cap, k["pool"] if paged else k["cont"],
                           zero_off if paged else H.to_dev(k["off"]), v["pool"] if paged else v["cont"],
                           zero_off if paged else H.to_dev(v["off"]), 1, k["dp"]["w_enc"], k["dp"]["w_dec"],
                           k["dp"]["m_rot"], k["dp"]["widths"], v["dp"]["w_enc"], v["dp"]["w_dec"], v["dp"]["m_rot"],
                           v["dp"]["widths"], 0.0, o, None, ws, status, k["params"].widths, v["params"].widths, **kw)
            torch.cuda.synchronize()
            res.append(o.cpu().numpy())
        assert np.array_equal(res[0], res[1])
    assert int(status.item()) == 0
    for name in ("k", "v"):
        c = S[name]
        g = gathered(name).reshape(n_seq, n_tiles, c["tb"])
        r = c["cont"].cpu().numpy().reshape(n_seq, n_tiles, c["tb"])
        assert np.array_equal(g[:, :5], r[:, :5])


@pytest.mark.parametrize("widths", ["all8", "all7", "v8_k1", "odd_mix"])
def test_tensor_core_attention_takes_any_width_profile(sp, widths):
    """The tensor-core kernels keep the value accumulators in tensor memory, block by block, so no width profile is
    special: 8-bit channels, three sub-fields per channel, one-bit keys with eight-bit values, and a mix with odd
    class sizes all run there and match the oracle."""
    wl = si.WORKLOADS["tiny"]
    cfg = sp.default_config()
    n = 700
    rng = np.random.default_rng(3)
    table = {"all8": (np.full(128, 8), np.full(128, 8)), "all7": (np.full(128, 7), np.full(128, 7)),
             "v8_k1": (np.ones(128, np.int64), np.full(128, 8)),
             "odd_mix": (rng.integers(0, 9, 128), rng.integers(0, 9, 128))}
    wk, wv = (np.asarray(w, np.uint8) for w in table[widths])
    S, caches = {}, {}
    for side, name, w in ((si.SIDE_K, "k", wk), (si.SIDE_V, "v", wv)):
        X = si.draw_unit(wl, 0, 0, side, 0, n_tokens=n)
        params = H.fit_params([X], 4.0, widths_override=w)
        off, total = H.cache_layout(params, 1, n)
        c = np.zeros(total, np.uint8)
        assert H.oracle_encode(params, side, X[None], [0], c, off) == 0
        S[name] = dict(X=X, params=params, off=off, total=total)
        caches[name] = c
    assert sp.attention_path(cfg, 1, 4, 1, S["k"]["params"].widths, S["v"]["params"].widths) == sp.PATH_TENSOR_CORE
    q = si.draw_queries(wl, 0, 0)
    ref_b, lse_b = _oracle_attention(4, q[None].astype(np.float64), [n], S["k"], S["v"], caches["k"], caches["v"])
    got, lse = _gpu_attention(sp, cfg, H.to_dev(q[None]), 1, 1, 4, [n], n, S["k"], S["v"], caches["k"], caches["v"])
    assert H.rel_err_per_vector(got[0], ref_b[0]) <= TOL
    assert np.abs(lse[0] - lse_b[0]).max() <= 2e-3


@pytest.mark.parametrize("width_group", [1, 64])
def test_pooled_allocation_is_bit_exact(sp, width_group):
    """spectra_alloc_bits_pooled against the oracle: budget pooled over the 8 heads of a layer, per channel and with
    one width per group of 64 coordinates (the paper's structure), several ratios, ties included."""
    rng = np.random.default_rng(23)
    H, layers = 8, 3
    v = ((np.arange(1, 129) ** -1.5)[None] * rng.uniform(0.02, 4.0, (layers * H, 1))).astype(np.float32)
    v[5, 40:60] = v[5, 40]                               # ties inside a head
    v[9] = v[8]                                          # and between heads
    v[17, 100:] = 0.0                                    # a dead tail
    cfg = sp.default_config(width_group=width_group)
    for ratio in (4.0, 8.0, 12.0):
        widths = torch.zeros((layers * H, 128), dtype=torch.uint8, device="cuda")
        sp.alloc_bits_pooled(cfg, torch.from_numpy(v).cuda(), layers * H, H, ratio, widths)
        torch.cuda.synchronize()
        got = widths.cpu().numpy()
        btot = ofit.total_bits(128, ratio)
        for l in range(layers):
            ref = ofit.alloc_bits_pooled(v[l * H:(l + 1) * H], btot, 8, width_group)
            assert np.array_equal(got[l * H:(l + 1) * H], ref), (width_group, ratio, l)
    rk, rv = sp.split_ratio(8.0, 0.25)
    assert (rk, rv) == ofit.split_ratio(8.0, 0.25) == (16.0, 8.0 / 1.5)


def test_paper_structure_allocation_end_to_end(sp):
    """The paper's allocation structure through the whole path: one width per group of 64 energy-ordered coordinates,
    the budget pooled over the KV heads of the layer (heads with little energy give their bits away, so tile sizes
    differ per head) and split between keys and values with kappa = 0.25 (Sec. 3.1-3.2, appendix on hyperparameters).
    Widths from the GPU equal the oracle's; encode, then attention on the tensor-core path, against the oracle."""
    base = si.WORKLOADS["llama1"]
    wl = dataclasses.replace(base, kv_heads=4, q_heads=16, n_fit=512)
    cfg = sp.default_config(width_group=64)
    n, Hk, G = 640, 4, 4
    head_scale = np.array([3.0, 1.0, 0.3, 0.05], np.float32)          # very unequal heads
    rk, rv = sp.split_ratio(8.0, 0.25)
    S = {}
    for side, name, ratio in ((si.SIDE_K, "k", rk), (si.SIDE_V, "v", rv)):
        X = H.draw_units(wl, 0, side, 1, n) * head_scale[:, None, None]
        fits = [ofit.fit_basis(X[h][:512].astype(np.float64), ofit.GAIN_SQRT) for h in range(Hk)]
        v_alloc = np.stack([f["v_alloc"] for f in fits]).astype(np.float32)
        ref_w = ofit.alloc_bits_pooled(v_alloc, ofit.total_bits(128, ratio), 8, 64)
        widths = torch.zeros((Hk, 128), dtype=torch.uint8, device="cuda")
        sp.alloc_bits_pooled(cfg, torch.from_numpy(v_alloc).cuda(), Hk, Hk, ratio, widths)
        torch.cuda.synchronize()
        assert np.array_equal(widths.cpu().numpy(), ref_w)
        assert len(set(ref_w.sum(axis=1))) > 1                         # the heads did get different budgets
        params = H.Params(np.stack([f["W_enc"] for f in fits]), np.stack([f["W_dec"] for f in fits]),
                          np.stack([f["m_rot"] for f in fits]), ref_w, 64)
        off, total = H.cache_layout(params, Hk, n)
        cache = torch.zeros(total, dtype=torch.uint8, device="cuda")
        st = _gpu_encode(sp, cfg, params, H.dev_params(params), side, H.to_dev(X).to(torch.bfloat16),
                         torch.zeros(Hk, dtype=torch.int32, device="cuda"), cache, H.to_dev(off))
        assert st == 0
        ref = np.zeros(total, np.uint8)
        assert H.oracle_encode(params, side, si.to_bf16_f32(X), [0] * Hk, ref, off) == 0
        got = cache.cpu().numpy()
        for u in range(Hk):
            bad, tot, dmax, mmax, _ = H.compare_coded_units(ref[off[u]:], got[off[u]:], int(params.tile_bytes[u]), n,
                                                            params.widths[u], 64, side)
            assert dmax <= 1 and mmax <= 1 and bad <= max(2, MISMATCH_RATE * tot)
        S[name] = dict(params=params, off=off, total=total, cache=got)
    assert sp.attention_path(cfg, Hk, wl.q_heads, Hk, S["k"]["params"].widths, S["v"]["params"].widths) == \
        sp.PATH_TENSOR_CORE
    q = si.draw_queries(wl, 0, 0)[:wl.q_heads]
    got, lse = _gpu_attention(sp, cfg, H.to_dev(q[None]), 1, Hk, wl.q_heads, [n], n, S["k"], S["v"], S["k"]["cache"],
                              S["v"]["cache"])
    K, V = S["k"], S["v"]
    ref, lref = oc.attention_units("B", q.reshape(Hk, G, 128).astype(np.float64), [n] * Hk, K["cache"], K["off"],
                                   K["params"].tile_bytes, V["cache"], V["off"], V["params"].tile_bytes,
                                   K["params"].w_dec, K["params"].m_rot, K["params"].widths, V["params"].w_dec,
                                   V["params"].m_rot, V["params"].widths, 64, 1.0 / np.sqrt(128.0))
    assert H.rel_err_per_vector(got[0].reshape(Hk, G, 128), ref) <= TOL
    assert np.abs(lse[0].reshape(Hk, G) - lref).max() <= 2e-3


@pytest.mark.parametrize("dt", ["f32", "bf16"])
def test_reconstruction_with_rotary_positions_matches_oracle(sp, dt):
    """Sec. 3.3, Mode A: keys are reconstructed and then rotated at their positions.  spectra_decode_rope against the
    oracle's reconstruct-then-rotate, two units with different starting positions, ragged length."""
    wl, S = _tiny_setup(sp, 8.0)
    cfg = sp.default_config()
    s = S["k"]
    params = s["params"]
    n, theta = 900, 500000.0
    pos0 = np.array([0, 4000], np.int32)
    ref_cache = np.zeros(s["total"], np.uint8)
    H.oracle_encode(params, si.SIDE_K, s["X"][None, :n], [0], ref_cache, s["off"])
    tb = int(params.tile_bytes[0])
    want = [oc.decode_unit_rope(ref_cache, tb, n, params.w_dec[0], params.m_rot[0], params.widths[0], 64, si.SIDE_K,
                                float(p0), theta) for p0 in pos0]
    n_pos = int(pos0.max()) + 1024
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * theta ** (-2.0 * np.arange(64, dtype=np.float64) / 128.0)[None]
    cos_t, sin_t = H.to_dev(np.cos(ang).astype(np.float32)), H.to_dev(np.sin(ang).astype(np.float32))
    dp = H.dev_params(params)
    cache2 = H.to_dev(np.concatenate([ref_cache, ref_cache]))
    off2 = H.to_dev(np.array([0, ref_cache.size], np.int64))
    tdt = torch.float32 if dt == "f32" else torch.bfloat16
    out = torch.full((2, 1024, 128), 7.0, dtype=tdt, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sp.decode_rope(cfg, cache2, off2, 2, 1, torch.tensor([n, n - 100], dtype=torch.int32, device="cuda"), n, dp["w_dec"],
                   dp["m_rot"], dp["widths"], out, 1024 * 128, 128, cos_t, sin_t, H.to_dev(pos0), status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    tol = TOL if dt == "f32" else TOL + 2.0 ** -8
    got = out.float().cpu().numpy()
    assert H.rel_err_per_vector(got[0, :n], want[0]) <= tol
    assert H.rel_err_per_vector(got[1, :n - 100], want[1][:n - 100]) <= tol
    assert (got[0, n:] == 7.0).all() and (got[1, n - 100:] == 7.0).all()


@pytest.mark.parametrize("n_fit", [300, 1000, 4096])
def test_fit_moments_on_tensor_cores_are_accurate_and_reproducible(sp, n_fit):
    """bf16 inputs take the tensor-core moments (S = X^T X in fp32 per 256-token chunk, fp64 across chunks, fixed
    order).  The sums left in the caller's workspace are compared with the fp64 sums of the same bf16 values (Sec. 3.1:
    the basis is fitted from the second moments of the calibration tokens), for ragged token counts and inputs with a
    mean; two calls give the same bits."""
    wl = si.WORKLOADS["llama1"]
    heads, n_all = 3, 4200
    X = np.stack([si.draw_unit(wl, 0, h, si.SIDE_K, 0, n_tokens=n_all) for h in range(heads)])
    X[1] += 0.75                                                     # a unit with a clear mean
    cfg = sp.default_config()
    xd = H.to_dev(X).to(torch.bfloat16)
    Xb = xd.float().cpu().numpy().astype(np.float64)                 # the values the kernel reads
    f32 = dict(dtype=torch.float32, device="cuda")
    outs = []
    for rep in range(2):
        w_enc, w_dec = (torch.zeros((heads, 128, 128), **f32) for _ in range(2))
        m_rot, var, lam = (torch.zeros((heads, 128), **f32) for _ in range(3))
        ws = torch.full((sp.fit_workspace_bytes(cfg, heads),), 0xAB, dtype=torch.uint8, device="cuda")   # dirty
        sp.fit_basis(cfg, xd, heads, n_fit, n_all * 128, 128, w_enc, w_dec, m_rot, var, lam, None, ws)
        torch.cuda.synchronize()
        outs.append((w_enc.cpu().numpy(), lam.cpu().numpy(), ws.cpu().numpy().copy()))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    moments = outs[0][2].view(np.float64).reshape(heads, 128 * 128 + 128)
    for h in range(heads):
        S_ref = Xb[h, :n_fit].T @ Xb[h, :n_fit]
        s_ref = Xb[h, :n_fit].sum(axis=0)
        S = moments[h, :128 * 128].reshape(128, 128)
        assert np.abs(S - S_ref).max() <= 2e-5 * np.abs(S_ref).max()
        assert np.abs(moments[h, 128 * 128:] - s_ref).max() <= 1e-5 * max(1.0, np.abs(s_ref).max())
        ref = ofit.fit_basis(Xb[h, :n_fit], ofit.GAIN_SQRT)
        assert np.abs(outs[0][1][h] - ref["lam"]).max() <= 2e-6 * ref["lam"][0]


@pytest.mark.parametrize("case", ["fitted_8x", "fitted_4x", "all8", "all7", "all1", "odd_mix", "gs32", "gs128", "misaligned",
                                  "one_group_empty"])
def test_reconstruction_without_unpacked_codes_on_every_layout(sp, case):
    """spectra_decode with no yhat output feeds the packed fields to the tensor cores (Sec. 3.3 Mode A reconstruction
    regrouped per scale group) for every unit that kernel can hold, and the element-wise kernel takes the rest in the
    same call (tiles above the slot, more than 192 strip positions, four scale groups, a source that is not 16-byte
    aligned).  Both sides, fp32 and bf16 outputs, two units (one ragged), against the oracle's reconstruction."""
    wl = si.WORKLOADS["tiny"]
    gs = {"gs32": 32, "gs128": 128}.get(case, 64)
    cfg = sp.default_config(scale_group=gs)
    rng = np.random.default_rng(17)
    n, n2 = 700, 389
    shift = 6 if case == "misaligned" else 0
    for side in (si.SIDE_K, si.SIDE_V):
        X = si.draw_unit(wl, 0, 0, side, 0, n_tokens=n)
        if case == "fitted_8x" or case == "gs32" or case == "gs128" or case == "misaligned":
            params = H.fit_params([X], 8.0, gs=gs)
        elif case == "fitted_4x":
            params = H.fit_params([X], 4.0, gs=gs)
        else:
            w = {"all8": np.full(128, 8), "all7": np.full(128, 7), "all1": np.ones(128, np.int64),
                 "odd_mix": rng.integers(0, 9, 128),
                 "one_group_empty": np.concatenate([rng.integers(1, 5, 64), np.zeros(64, np.int64)])}[case]
            params = H.fit_params([X], 4.0, gs=gs, widths_override=np.asarray(w, np.uint8))
        tb = int(params.tile_bytes[0])
        off = np.array([0, 6 * tb], np.int64)                      # two units of six tiles each
        ref = np.zeros(12 * tb, np.uint8)
        assert H.oracle_encode(params, side, X[None, :n], [0], ref, off[:1]) == 0
        assert H.oracle_encode(params, side, X[None, 100:100 + n2], [0], ref, off[1:]) == 0
        want = [oc.decode_unit(ref[off[u]:], tb, m, params.w_dec[0], params.m_rot[0], params.widths[0], gs, side)[1]
                for u, m in ((0, n), (1, n2))]
        dp = H.dev_params(params)
        cache_dev = torch.zeros(ref.size + 16, dtype=torch.uint8, device="cuda")
        cache_dev[shift:shift + ref.size] = H.to_dev(ref)
        for dt in (torch.float32, torch.bfloat16):
            out = torch.full((2, 768, 128), 7.0, dtype=dt, device="cuda")
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            sp.decode(cfg, side, cache_dev[shift:], H.to_dev(off), 2, 1, torch.tensor([n, n2], dtype=torch.int32, device="cuda"),
                      n, dp["w_dec"], dp["m_rot"], dp["widths"], out, None, 768 * 128, 128, status_word=status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            tol = TOL if dt == torch.float32 else TOL + 2.0 ** -8
            got = out.float().cpu().numpy()
            assert H.rel_err_per_vector(got[0, :n], want[0]) <= tol
            assert H.rel_err_per_vector(got[1, :n2], want[1]) <= tol
            assert (got[0, n:] == 7.0).all() and (got[1, n2:] == 7.0).all()


@pytest.mark.parametrize("skew", [16, 8, 1])
def test_reconstruction_into_outputs_of_any_alignment(sp, skew):
    """The packed-field reconstruction stores 32 bytes per instruction where the output allows it; an output that
    starts `skew` elements into a 32-byte-aligned buffer takes the 16-byte or the element-wise stores instead.  All of
    them write the same values, and nothing outside the unit's tokens."""
    wl = si.WORKLOADS["tiny"]
    cfg = sp.default_config()
    n = 300
    for side in (si.SIDE_K, si.SIDE_V):
        X = si.draw_unit(wl, 0, 0, side, 0, n_tokens=n)
        params = H.fit_params([X], 8.0)
        tb = int(params.tile_bytes[0])
        ref = np.zeros(3 * tb, np.uint8)
        assert H.oracle_encode(params, side, X[None, :n], [0], ref, np.zeros(1, np.int64)) == 0
        dp = H.dev_params(params)
        cache_dev = H.to_dev(ref)
        off = H.to_dev(np.zeros(1, np.int64))
        n_dev = torch.tensor([n], dtype=torch.int32, device="cuda")
        for dt in (torch.bfloat16, torch.float32):
            outs = []
            for s in (0, skew):
                buf = torch.full((384 * 128 + 64,), 7.0, dtype=dt, device="cuda")
                out = buf[s:s + 384 * 128].view(1, 384, 128)
                assert out.data_ptr() % 32 == (s * buf.element_size()) % 32
                status = torch.zeros(1, dtype=torch.int32, device="cuda")
                sp.decode(cfg, side, cache_dev, off, 1, 1, n_dev, n, dp["w_dec"], dp["m_rot"], dp["widths"], out, None,
                          384 * 128, 128, status_word=status)
                torch.cuda.synchronize()
                assert int(status.item()) == 0
                full = buf.float().cpu().numpy()
                assert (full[:s] == 7.0).all() and (full[s + n * 128:] == 7.0).all()
                outs.append(full[s:s + n * 128])
            assert np.array_equal(outs[0], outs[1])


def test_quotients_from_a_shared_reciprocal_equal_the_division(sp):
    """The bulk encoder's L_b / R16 (one reciprocal, fused multiply-add corrections) against the IEEE division for
    every positive finite fp16 R16 and every width: not one bit may differ, or its codes would not be the oracle's."""
    bad = torch.full((1,), -1, dtype=torch.int64, device="cuda")
    sp.selftest_quotients(bad)
    torch.cuda.synchronize()
    assert int(bad.item()) == 0
