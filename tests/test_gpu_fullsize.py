"""Parity at the workloads' full context lengths, in the launch configuration bench.py times (the harness the
benchmark uses), on sampled units the oracle can compute one by one.

Both sides get the same transforms and widths (fitted by the oracle from the same raw vectors); the GPU encodes
every unit of the layer, appends one token per sequence and attends; the oracle does the same for the sampled
(sequence, kv-head) units from the raw vectors alone.  Checked: EVERY token of the sampled units, code by code and
metadata word by word (codes differ by one level at most, in at most 1e-4 of the active entries, tokens whose
metadata differ included; metadata differ by one fp16 step at most); the attention output over the bytes the GPU
itself encoded (the oracle attends over a copy of those bytes) and over the oracle's bytes (2e-3, max |diff| /
max |oracle| per vector).  A second step then goes through the fused call the benchmark times
(spectra_decode_step): the token it appended is compared code by code with the oracle's encode, and its output
with the oracle's attention over the very bytes the GPU holds after the step.  The encode sweep (1K to 128K
appended tokens at 4x, 8x and 12x) is compared the same way, every token.
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

MISMATCH_RATE = 1e-4      # of active entries, +-1 level only

CASES = {
    # name: (workload, batch used here, sampled (sequence, kv-head) units)
    "llama1_4x_32k": ("llama1", 1, [(0, 0), (0, 5)]),
    "llama32_8x_32k_batch8": ("llama32", 8, [(0, 0), (3, 5), (7, 7)]),
    "qwen28_12x_64k_batch16": ("qwen28", 16, [(0, 1), (9, 3), (15, 0)]),
    "long_8x_128k": ("long128k", 1, [(0, 2)]),
    "batch32_8x_32k": ("batch32", 32, [(0, 0), (17, 3), (31, 7)]),
}


@pytest.mark.parametrize("case", list(CASES))
def test_full_context_decode_step_matches_oracle(case):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2608_07915_b200 as sp
    from paper_2608_07915_b200 import harness
    name, batch, sampled = CASES[case]
    wl = si.WORKLOADS[name]
    Hk, G, d, N = wl.kv_heads, wl.group, wl.head_dim, wl.n_tokens
    model = harness.CodedModelCache(wl, layers=1, batch=batch, extra_tokens=128)
    # raw vectors (generator output, not codec output): fit tokens of sequence 0 for every head, and the sampled units
    params, raw = {}, {}
    for side in (si.SIDE_K, si.SIDE_V):
        x = model.draw_layer_side(0, side)                                     # [batch, H, N, d]
        fits = [ofit.fit_basis(x[0, h, :wl.n_fit].float().cpu().numpy().astype(np.float64), ofit.GAIN_SQRT)
                for h in range(Hk)]
        widths = np.stack([ofit.alloc_bits(f["v_alloc"].astype(np.float32), ofit.total_bits(d, wl.ratio))
                           for f in fits])
        params[(0, side)] = dict(w_enc=np.stack([f["W_enc"] for f in fits]), w_dec=np.stack([f["W_dec"] for f in fits]),
                                 m_rot=np.stack([f["m_rot"] for f in fits]), widths=widths)
        for (s, h) in sampled:
            raw[(side, s, h)] = x[s, h].float().cpu().numpy()
        del x
    model.build(params_override=params)          # same generator seeds: the harness redraws the same vectors
    assert int(model.status.item()) == 0
    # one decode step on the GPU
    gen = torch.Generator(device="cuda").manual_seed(99)
    q = torch.randn((1, batch, wl.q_heads, d), generator=gen, device="cuda").to(torch.bfloat16)
    nk = torch.randn((1, batch * Hk, d), generator=gen, device="cuda").to(torch.bfloat16)
    nv = torch.randn((1, batch * Hk, d), generator=gen, device="cuda").to(torch.bfloat16)
    out = torch.zeros((1, batch, wl.q_heads, d), dtype=torch.float32, device="cuda")
    # the decode step, in the harness's order: lengths grow, K and V appends, attention
    model.seq_len += 1
    model.append(0, nk[0], nv[0])
    torch.cuda.synchronize()
    assert int(model.status.item()) == 0
    qh = q[0].float().cpu().numpy().reshape(batch, Hk, G, d).astype(np.float64)
    new = {si.SIDE_K: nk[0].float().cpu().numpy(), si.SIDE_V: nv[0].float().cpu().numpy()}
    n_tiles = (N + 1 + 127) // 128
    oracle_caches, gpu_bytes = {}, {}
    stats = {si.SIDE_K: [0, 0], si.SIDE_V: [0, 0]}
    for (s, h) in sampled:
        u = s * Hk + h
        caches = {}
        for side in (si.SIDE_K, si.SIDE_V):
            P = params[(0, side)]
            pr = H.Params(P["w_enc"][[h]], P["w_dec"][[h]], P["m_rot"][[h]], P["widths"][[h]], 64)
            tb = int(pr.tile_bytes[0])
            c = np.zeros(n_tiles * tb, np.uint8)
            xs = np.concatenate([raw[(side, s, h)], new[side][u][None]], axis=0)
            assert H.oracle_encode(pr, side, xs[None], [0], c, np.zeros(1, np.int64)) == 0
            caches[side] = (pr, tb, c)
            # the GPU's bytes for this unit, every token: codes within one level, metadata within one fp16 step
            ls = model.side[0][side]
            a = int(ls.unit_offset_host[u])
            g = ls.cache[a:a + n_tiles * tb].cpu().numpy()
            bad, tot, dmax, mmax, _ = H.compare_coded_units(c, g, tb, N + 1, pr.widths[0], 64, side)
            assert dmax <= 1 and mmax <= 1, (case, side, dmax, mmax)
            stats[side][0] += bad; stats[side][1] += tot
            gpu_bytes[(s, h, side)] = g
        oracle_caches[(s, h)] = caches
    for side in (si.SIDE_K, si.SIDE_V):
        assert stats[side][0] <= MISMATCH_RATE * stats[side][1], (case, side, stats[side])
    # attention over the bytes the GPU encoded itself: the oracle attends over a copy of the same bytes
    model.attend(0, q[0], out[0])
    torch.cuda.synchronize()
    assert int(model.status.item()) == 0
    got = out[0].cpu().numpy().reshape(batch, Hk, G, d)
    for (s, h) in sampled:
        (pk, tbk, _), (pv, tbv, _) = oracle_caches[(s, h)][si.SIDE_K], oracle_caches[(s, h)][si.SIDE_V]
        ref, _ = oc.attention_units("B", qh[s, h][None], [N + 1], gpu_bytes[(s, h, si.SIDE_K)], [0], [tbk],
                                    gpu_bytes[(s, h, si.SIDE_V)], [0], [tbv], pk.w_dec, pk.m_rot, pk.widths, pv.w_dec,
                                    pv.m_rot, pv.widths, 64, 1.0 / np.sqrt(128.0))
        assert H.rel_err_per_vector(got[s, h], ref[0]) <= TOL, (case, "gpu bytes", s, h)
    # and over the oracle's bytes, uploaded into the sampled units' caches
    for (s, h) in sampled:
        u = s * Hk + h
        for side in (si.SIDE_K, si.SIDE_V):
            pr, tb, c = oracle_caches[(s, h)][side]
            ls = model.side[0][side]
            a = int(ls.unit_offset_host[u])
            ls.cache[a:a + n_tiles * tb].copy_(torch.from_numpy(c).cuda())
    model.attend(0, q[0], out[0])
    torch.cuda.synchronize()
    assert int(model.status.item()) == 0
    got = out[0].cpu().numpy().reshape(batch, Hk, G, d)
    for (s, h) in sampled:
        caches = oracle_caches[(s, h)]
        (pk, tbk, ck), (pv, tbv, cv) = caches[si.SIDE_K], caches[si.SIDE_V]
        ref, _ = oc.attention_units("B", qh[s, h][None], [N + 1], ck, [0], [tbk], cv, [0], [tbv], pk.w_dec, pk.m_rot,
                                    pk.widths, pv.w_dec, pv.m_rot, pv.widths, 64, 1.0 / np.sqrt(128.0))
        # bf16 queries on the GPU side are exactly the fp32 values the oracle used
        assert H.rel_err_per_vector(got[s, h], ref[0]) <= TOL, (case, s, h)
    # ---- reconstruction of the whole layer in the launch bench.py times (every unit, bf16 out): the sampled units, which
    #      hold the oracle's bytes now, against the oracle's reconstruction; every token
    U = batch * Hk
    n_rec = N + 1
    if U * n_rec * d * 2 <= (6 << 30):
        recon = torch.empty((U, n_rec, d), dtype=torch.bfloat16, device="cuda")
        for side in (si.SIDE_K, si.SIDE_V):
            ls = model.side[0][side]
            sp.decode(model.cfg, side, ls.cache, ls.unit_offset, U, Hk, torch.full((U,), n_rec, dtype=torch.int32, device="cuda"),
                      n_rec, ls.w_dec, ls.m_rot, ls.widths, recon, None, n_rec * d, d, status_word=model.status)
            torch.cuda.synchronize()
            assert int(model.status.item()) == 0
            for (s, h) in sampled:
                pr, tb, c = oracle_caches[(s, h)][side]
                _, want = oc.decode_unit(c, tb, n_rec, pr.w_dec[0], pr.m_rot[0], pr.widths[0], 64, side, want_yhat=False)
                got_r = recon[s * Hk + h].float().cpu().numpy()
                assert H.rel_err_per_vector(got_r, want) <= TOL + 2.0 ** -8, (case, "reconstruction", side, s, h)
        del recon
    # ---- a second step through the fused call (the one bench.py times)
    q2 = torch.randn((batch, wl.q_heads, d), generator=gen, device="cuda").to(torch.bfloat16)
    nk2 = torch.randn((batch * Hk, d), generator=gen, device="cuda").to(torch.bfloat16)
    nv2 = torch.randn((batch * Hk, d), generator=gen, device="cuda").to(torch.bfloat16)
    out2 = torch.zeros((batch, wl.q_heads, d), dtype=torch.float32, device="cuda")
    model.pos0 += 1
    model.seq_len += 1
    model.step_layer(0, q2, nk2, nv2, out2)
    torch.cuda.synchronize()
    assert int(model.status.item()) == 0
    got2 = out2.cpu().numpy().reshape(batch, Hk, G, d)
    qh2 = q2.float().cpu().numpy().reshape(batch, Hk, G, d).astype(np.float64)
    new2 = {si.SIDE_K: nk2.float().cpu().numpy(), si.SIDE_V: nv2.float().cpu().numpy()}
    n2 = N + 2
    n_tiles2 = (n2 + 127) // 128
    for (s, h) in sampled:
        u = s * Hk + h
        held = {}
        for side in (si.SIDE_K, si.SIDE_V):
            pr, tb, _ = oracle_caches[(s, h)][side]
            ls = model.side[0][side]
            a = int(ls.unit_offset_host[u])
            g = ls.cache[a:a + n_tiles2 * tb].cpu().numpy()
            # the appended token (position N + 1): the oracle encodes the same vector; ties differ by one level at most
            one = np.zeros(tb, np.uint8)
            slot = (N + 1) % 128
            assert H.oracle_encode(pr, side, new2[side][u][None, None], [slot], one, np.zeros(1, np.int64)) == 0
            cr, lr, rr = oc.unpack_token(one, pr.widths[0], 64, side, slot)
            tile = (N + 1) // 128
            cg, lg, rg = oc.unpack_token(g[tile * tb:(tile + 1) * tb], pr.widths[0], 64, side, slot)
            assert np.abs(cr.astype(np.int64) - cg.astype(np.int64)).max() <= 1
            held[side] = (pr, tb, g)
        (pk, tbk, ck), (pv, tbv, cv) = held[si.SIDE_K], held[si.SIDE_V]
        ref, _ = oc.attention_units("B", qh2[s, h][None], [n2], ck, [0], [tbk], cv, [0], [tbv], pk.w_dec, pk.m_rot,
                                    pk.widths, pv.w_dec, pv.m_rot, pv.widths, 64, 1.0 / np.sqrt(128.0))
        assert H.rel_err_per_vector(got2[s, h], ref[0]) <= TOL, (case, "fused", s, h)


@pytest.mark.parametrize("ratio", [4.0, 8.0, 12.0])
@pytest.mark.parametrize("n_tokens", [1024, 16384, 131072])
def test_encode_sweep_matches_oracle(ratio, n_tokens):
    """The encode sweep of the long-context configuration: n_tokens bf16 vectors appended to one head (the tiny
    configuration's recipe, both sides) at 4x, 8x and 12x; every token of the packed result against the oracle."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2608_07915_b200 as sp
    wl = dataclasses.replace(si.WORKLOADS["tiny"], dtype="bf16")
    cfg = sp.default_config()
    for side in (si.SIDE_K, si.SIDE_V):
        x = si.draw_unit_torch(wl, 0, 0, side, 1, n_tokens, "cuda")[0]                  # [n, d] bf16
        xf = x.float().cpu().numpy()
        pr = H.fit_params([xf[:1024]], ratio)
        tb = int(pr.tile_bytes[0])
        n_tiles = (n_tokens + 127) // 128
        ref = np.zeros(n_tiles * tb, np.uint8)
        assert H.oracle_encode(pr, side, xf[None], [0], ref, np.zeros(1, np.int64)) == 0
        dp = H.dev_params(pr)
        cache = torch.full((n_tiles * tb,), 0xAA, dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        sp.encode(cfg, side, x, 0, 1, 1, torch.zeros(1, dtype=torch.int32, device="cuda"), n_tokens, n_tokens * 128,
                  128, dp["w_enc"], dp["m_rot"], dp["widths"], cache, torch.zeros(1, dtype=torch.int64, device="cuda"),
                  status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        bad, tot, dmax, mmax, _ = H.compare_coded_units(ref, cache.cpu().numpy(), tb, n_tokens, pr.widths[0], 64, side)
        assert dmax <= 1 and mmax <= 1, (ratio, n_tokens, side, dmax, mmax)
        # a single short run may hold one tie where the rate allows a fraction of one: allow that one
        assert bad <= max(1, MISMATCH_RATE * tot), (ratio, n_tokens, side, bad, tot)
