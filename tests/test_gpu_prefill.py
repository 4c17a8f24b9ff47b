"""GPU parity of the many-query path (Sec. 3.3, Mode A for a chunk of queries): reconstruction into paged bf16 pools
(spectra_decode_paged) and causal attention over them (spectra_prefill_attention), against oracle/prefill.py.

Tolerances.  The kernel reads bf16 keys and values (the storage the reconstruction is written in), rounds the
probabilities to bf16 before P V, normalises with their fp32 sum and rounds the output to bf16:
  * the attention kernel alone, on seeded bf16 pools, against the oracle on the same values: a weight is off by at
    most 2^-9 relative (the bf16 rounding of its probability; the sum is not rounded) and the output's rounding adds
    2^-9 of its size; errors of independent tokens do not add up coherently, so 1e-2 of a vector's largest entry
    bounds what remains (measured: a few 1e-3), and lse, which only sees the sum, stays within 5e-3;
  * the whole path from coded bytes against the oracle's Mode A in fp64: the bf16 storage (2^-9 per entry) and the
    reconstruction's own 2e-3 enter the keys, which moves a score by up to about 1e-2, hence 3e-2 on outputs and lse.
"""
import dataclasses

import numpy as np
import pytest

import spectra_inputs as si
from oracle import codec as oc
from oracle import prefill as opf
from tests import helpers as H

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL_SAME_STORAGE = 1e-2
TOL_LSE = 5e-3
TOL_F64_STORAGE = 3e-2


@pytest.fixture(scope="module")
def sp():
    if not torch.cuda.is_available():
        pytest.skip("needs a GPU")
    import paper_2608_07915_b200 as sp_
    sp_.lib()
    return sp_


def _setup(n_seq, kv_lens, ratio=4.0):
    base = si.WORKLOADS["llama1"]
    wl = dataclasses.replace(base, kv_heads=2, q_heads=2 * base.group, n_fit=512)
    n_tok = max(kv_lens)
    S = {}
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        X = H.draw_units(wl, 0, side, n_seq, max(n_tok, 512))
        params = H.fit_params([X[h][:512] for h in range(wl.kv_heads)], ratio)
        n_units = n_seq * wl.kv_heads
        off, total = H.cache_layout(params, n_units, n_tok)
        cache = np.zeros(total, np.uint8)
        for u in range(n_units):
            p = u % wl.kv_heads
            one = H.Params(params.w_enc[[p]], params.w_dec[[p]], params.m_rot[[p]], params.widths[[p]], 64)
            H.oracle_encode(one, side, X[u][None, :kv_lens[u // wl.kv_heads]], [0], cache[off[u]:], np.zeros(1, np.int64))
        S[name] = dict(params=params, off=off, cache=cache)
    return wl, S


def _paged_reconstruction(sp, wl, S, n_seq, kv_lens, rng, fill):
    """Both sides into bf16 pools through one shuffled page table; unused slots keep `fill`."""
    cfg = sp.default_config()
    n_units = n_seq * wl.kv_heads
    max_len = max(kv_lens)
    tiles = (max_len + 127) // 128
    n_pages = n_units * tiles + 3
    table = rng.permutation(n_pages)[:n_units * tiles].astype(np.int32).reshape(n_units, tiles)
    table_d = H.to_dev(table)
    n_tok_d = H.to_dev(np.array([kv_lens[u // wl.kv_heads] for u in range(n_units)], np.int32))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    pools = {}
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        s = S[name]
        dp = H.dev_params(s["params"])
        pool = torch.full((n_pages, 128, 128), fill, dtype=torch.bfloat16, device="cuda")
        sp.decode_paged(cfg, side, H.to_dev(s["cache"]), H.to_dev(s["off"]), n_units, wl.kv_heads, n_tok_d, max_len,
                        dp["w_dec"], dp["m_rot"], dp["widths"], pool, 128 * 128, 128, table_d, tiles,
                        status_word=status)
        pools[name] = pool
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return pools, table, table_d, tiles, n_pages


def test_paged_reconstruction_matches_oracle(sp):
    """spectra_decode_paged: every token lands in the page its table names, at its slot; nothing else is written."""
    n_seq, kv_lens = 2, [350, 227]
    wl, S = _setup(n_seq, kv_lens, 8.0)
    pools, table, _, tiles, n_pages = _paged_reconstruction(sp, wl, S, n_seq, kv_lens, np.random.default_rng(1), 7.0)
    for side, name in ((si.SIDE_K, "k"), (si.SIDE_V, "v")):
        s = S[name]
        got = pools[name].float().cpu().numpy()
        written = np.zeros((n_pages, 128), bool)
        for u in range(n_seq * wl.kv_heads):
            p, n = u % wl.kv_heads, kv_lens[u // wl.kv_heads]
            _, want = oc.decode_unit(s["cache"][s["off"][u]:], int(s["params"].tile_bytes[p]), n, s["params"].w_dec[p],
                                     s["params"].m_rot[p], s["params"].widths[p], 64, side)
            for t in range((n + 127) // 128):
                m = min(128, n - 128 * t)
                assert H.rel_err_per_vector(got[table[u, t], :m], want[128 * t:128 * t + m]) <= 2e-3 + 2.0 ** -8
                written[table[u, t], :m] = True
        assert (got[~written] == 7.0).all()


SHAPES = [([200, 77], 150), ([0], 1000), ([1000], 1), ([127, 128], 129)]


@pytest.mark.parametrize("Hkv,G", [(2, 4), (4, 7), (3, 1)], ids=["gqa4", "gqa7", "mha"])
@pytest.mark.parametrize("pos0,n_new", SHAPES)
def test_prefill_attention_kernel_on_seeded_pools(sp, pos0, n_new, Hkv, G):
    """The attention kernel alone: seeded bf16 keys and values laid out through a shuffled page table, every slot past
    a sequence's end NaN, against the oracle's causal attention on the same bf16 values, row by row (ragged chunk
    ends, a chunk that starts mid-tile, a single query, the diagonal crossing two tiles)."""
    n_seq, d = len(pos0), 128
    if (Hkv, G) != (2, 4) and n_new == 1000:
        pytest.skip("the long chunk is covered at one head shape")
    Hq = Hkv * G
    kv_lens = [p + n_new for p in pos0]
    tiles = (max(kv_lens) + 127) // 128
    n_units = n_seq * Hkv
    n_pages = n_units * tiles + 3
    rng = np.random.default_rng(11)
    table = rng.permutation(n_pages)[:n_units * tiles].astype(np.int32).reshape(n_units, tiles)
    K = H.to_dev((rng.standard_normal((n_units, tiles * 128, d)) * 1.2).astype(np.float32)).to(torch.bfloat16)
    V = H.to_dev((rng.standard_normal((n_units, tiles * 128, d)) * 2.0 + 0.5).astype(np.float32)).to(torch.bfloat16)
    kp = torch.full((n_pages, 128, d), float("nan"), dtype=torch.bfloat16, device="cuda")
    vp = torch.full((n_pages, 128, d), float("nan"), dtype=torch.bfloat16, device="cuda")
    for u in range(n_units):
        n = kv_lens[u // Hkv]
        for t in range((n + 127) // 128):
            m = min(128, n - 128 * t)
            kp[table[u, t], :m] = K[u, 128 * t:128 * t + m]
            vp[table[u, t], :m] = V[u, 128 * t:128 * t + m]
    q = H.to_dev((rng.standard_normal((n_seq, n_new, Hq, d)) * 1.5).astype(np.float32)).to(torch.bfloat16)
    out = torch.full((n_seq, n_new, Hq, d), 5.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((n_seq, n_new, Hq), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    scale = 1.0 / np.sqrt(d)
    strides = (n_new * Hq * d, Hq * d, d)
    sp.prefill_attention(q, kp, vp, n_pages, 128 * d, d, H.to_dev(table), tiles, n_seq, Hkv, Hq,
                         H.to_dev(np.array(pos0, np.int32)), n_new, strides, scale, out, strides, lse, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got, got_lse = out.float().cpu().numpy(), lse.cpu().numpy()
    assert np.isfinite(got).all() and np.isfinite(got_lse).all()
    Kh, Vh, qh = (x.float().cpu().numpy().astype(np.float64) for x in (K, V, q))
    worst = 0.0
    for b in range(n_seq):
        for kh in range(Hkv):
            u = b * Hkv + kh
            ref, lref = opf.causal_attention(qh[b, :, kh * G:(kh + 1) * G], Kh[u, :kv_lens[b]], Vh[u, :kv_lens[b]], pos0[b], scale)
            worst = max(worst, H.rel_err_per_vector(got[b, :, kh * G:(kh + 1) * G], ref))
            assert np.abs(got_lse[b, :, kh * G:(kh + 1) * G] - lref).max() <= TOL_LSE
    assert worst <= TOL_SAME_STORAGE, worst


@pytest.mark.parametrize("pos0,n_new", SHAPES[:2])
def test_reconstruct_then_attend_matches_oracle_mode_a(sp, pos0, n_new):
    """The whole many-query path: coded caches -> spectra_decode_paged (bf16 pools, NaN where nothing is written) ->
    spectra_prefill_attention, against the oracle's Mode A in fp64 from the same coded bytes."""
    n_seq = len(pos0)
    kv_lens = [p + n_new for p in pos0]
    wl, S = _setup(n_seq, kv_lens)
    rng = np.random.default_rng(3)
    pools, table, table_d, tiles, n_pages = _paged_reconstruction(sp, wl, S, n_seq, kv_lens, rng, float("nan"))
    Hq, G = wl.q_heads, wl.group
    q = (rng.standard_normal((n_seq, n_new, Hq, 128)) * 1.5).astype(np.float32)
    q_d = H.to_dev(q).to(torch.bfloat16)
    q_used = q_d.float().cpu().numpy().astype(np.float64)          # the queries are bf16 inputs: both sides read these
    out = torch.full((n_seq, n_new, Hq, 128), 5.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((n_seq, n_new, Hq), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    scale = 1.0 / np.sqrt(128.0)
    strides = (n_new * Hq * 128, Hq * 128, 128)
    sp.prefill_attention(q_d, pools["k"], pools["v"], n_pages, 128 * 128, 128, table_d, tiles, n_seq, wl.kv_heads, Hq,
                         H.to_dev(np.array(pos0, np.int32)), n_new, strides, scale, out, strides, lse, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = out.float().cpu().numpy()
    got_lse = lse.cpu().numpy()
    assert np.isfinite(got).all() and np.isfinite(got_lse).all()
    K, V = S["k"], S["v"]
    worst64 = 0.0
    for b in range(n_seq):
        for kh in range(wl.kv_heads):
            u = b * wl.kv_heads + kh
            ref64, lref64 = opf.prefill_mode_a(
                q_used[b, :, kh * G:(kh + 1) * G], pos0[b], K["cache"][K["off"][u]:], int(K["params"].tile_bytes[kh]),
                V["cache"][V["off"][u]:], int(V["params"].tile_bytes[kh]), K["params"].w_dec[kh], K["params"].m_rot[kh],
                K["params"].widths[kh], V["params"].w_dec[kh], V["params"].m_rot[kh], V["params"].widths[kh], 64, scale)
            worst64 = max(worst64, H.rel_err_per_vector(got[b, :, kh * G:(kh + 1) * G], ref64))
            assert np.abs(got_lse[b, :, kh * G:(kh + 1) * G] - lref64).max() <= TOL_F64_STORAGE
    assert worst64 <= TOL_F64_STORAGE, worst64


def test_prefill_attention_argument_checks(sp):
    q = torch.zeros((1, 4, 2, 128), dtype=torch.bfloat16, device="cuda")
    pool = torch.zeros((2, 128, 128), dtype=torch.bfloat16, device="cuda")
    pos = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = (4 * 2 * 128, 2 * 128, 128)
    with pytest.raises(sp.SpectraError):       # three query heads over two KV heads
        sp.prefill_attention(q, pool, pool, 2, 128 * 128, 128, None, 1, 1, 2, 3, pos, 4, st, 0.1, q, st)
    with pytest.raises(sp.SpectraError):       # a token stride that is not a multiple of 8 elements
        sp.prefill_attention(q, pool, pool, 2, 128 * 128, 132, None, 1, 1, 2, 2, pos, 4, st, 0.1, q, st)
    with pytest.raises(sp.SpectraError):       # no table and no pages-per-unit
        sp.prefill_attention(q, pool, pool, 2, 128 * 128, 128, None, 0, 1, 2, 2, pos, 4, st, 0.1, q, st)
    sp.prefill_attention(q, pool, pool, 2, 128 * 128, 128, None, 1, 0, 2, 2, pos, 4, st, 0.1, q, st)   # nothing to do
    torch.cuda.synchronize()


def test_prefill_attention_at_the_benchmarked_size_on_sampled_rows(sp):
    """The launch bench.py times (one 32768-token chunk, 32 query / 8 KV heads, seeded random bf16 pools): sampled
    (row, head) outputs against the oracle's causal attention on the same bf16 values, row by row.  Rows at the start,
    at tile and block edges, in the middle and at the end; every KV group is sampled."""
    n_new, Hq, Hkv, d = 32768, 32, 8, 128
    tiles = n_new // 128
    n_pages = Hkv * tiles
    gen = torch.Generator(device="cuda").manual_seed(99)
    kp = torch.randn((n_pages, 128, d), generator=gen, device="cuda").to(torch.bfloat16)
    vp = torch.randn((n_pages, 128, d), generator=gen, device="cuda").to(torch.bfloat16)
    q = torch.randn((1, n_new, Hq, d), generator=gen, device="cuda").to(torch.bfloat16)
    out = torch.empty_like(q)
    lse = torch.zeros((1, n_new, Hq), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    strides = (n_new * Hq * d, Hq * d, d)
    scale = 1.0 / np.sqrt(d)
    sp.prefill_attention(q, kp, vp, n_pages, 128 * d, d, None, tiles, 1, Hkv, Hq, torch.zeros(1, dtype=torch.int32, device="cuda"),
                         n_new, strides, scale, out, strides, lse, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rows = [0, 1, 127, 128, 255, 256, 257, 4095, 16384, 20000, 32639, 32640, 32767]
    heads = [0, 5, 10, 15, 17, 22, 27, 31]                          # one per KV group
    worst = 0.0
    for h in heads:
        kh = h // (Hq // Hkv)
        K = kp[kh * tiles:(kh + 1) * tiles].reshape(-1, d).float().cpu().numpy().astype(np.float64)
        V = vp[kh * tiles:(kh + 1) * tiles].reshape(-1, d).float().cpu().numpy().astype(np.float64)
        for i in rows:
            qi = q[0, i, h].float().cpu().numpy().astype(np.float64)[None, None]
            ref, lref = opf.causal_attention(qi, K, V, i, scale)
            got = out[0, i, h].float().cpu().numpy()
            worst = max(worst, H.rel_err_per_vector(got[None], ref[0]))
            assert abs(float(lse[0, i, h].item()) - lref[0, 0]) <= TOL_LSE
    assert worst <= TOL_SAME_STORAGE, worst


def test_paged_reconstruction_with_rotary_positions(sp):
    """spectra_decode_paged with the position rotation of keys (Sec. 3.3: applied after reconstruction), fp32 pages."""
    n_seq, kv_lens = 1, [300]
    wl, S = _setup(n_seq, kv_lens, 8.0)
    cfg = sp.default_config()
    s = S["k"]
    n_units, n, theta = wl.kv_heads, 300, 500000.0
    tiles = 3
    table = np.array([[4, 0, 2], [1, 5, 3]], np.int32)
    pos0 = np.array([0, 1000], np.int32)
    n_pos = 1000 + 384
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * theta ** (-2.0 * np.arange(64, dtype=np.float64) / 128.0)[None]
    cos_t, sin_t = H.to_dev(np.cos(ang).astype(np.float32)), H.to_dev(np.sin(ang).astype(np.float32))
    dp = H.dev_params(s["params"])
    pool = torch.full((6, 128, 128), 7.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sp.decode_paged(cfg, si.SIDE_K, H.to_dev(s["cache"]), H.to_dev(s["off"]), n_units, wl.kv_heads,
                    H.to_dev(np.full(n_units, n, np.int32)), n, dp["w_dec"], dp["m_rot"], dp["widths"], pool, 128 * 128, 128,
                    H.to_dev(table), tiles, position0=H.to_dev(pos0), rope_cos=cos_t, rope_sin=sin_t, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = pool.cpu().numpy()
    for u in range(n_units):
        want = oc.decode_unit_rope(s["cache"][s["off"][u]:], int(s["params"].tile_bytes[u]), n, s["params"].w_dec[u],
                                   s["params"].m_rot[u], s["params"].widths[u], 64, si.SIDE_K, float(pos0[u]), theta)
        for t in range(tiles):
            m = min(128, n - 128 * t)
            assert H.rel_err_per_vector(got[table[u, t], :m], want[128 * t:128 * t + m]) <= 2e-3
            assert (got[table[u, t], m:] == 7.0).all()
    with pytest.raises(sp.SpectraError):                              # positions are for keys
        sp.decode_paged(cfg, si.SIDE_V, H.to_dev(s["cache"]), H.to_dev(s["off"]), n_units, wl.kv_heads,
                        H.to_dev(np.full(n_units, n, np.int32)), n, dp["w_dec"], dp["m_rot"], dp["widths"], pool, 128 * 128,
                        128, H.to_dev(table), tiles, rope_cos=cos_t, rope_sin=sin_t)
