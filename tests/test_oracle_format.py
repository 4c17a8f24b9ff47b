"""Pins for the oracle's fp16 rounding, sub-field split, tile layout, packer and quantiser (CPU only)."""
import itertools
import os

import numpy as np
import pytest

from oracle import codec, fit

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- fp16 directed rounding

def test_half_roundtrip_every_finite_value():
    bits = np.arange(0, 0x7C00, dtype=np.uint16)
    for sign in (0, 0x8000):
        b = (bits | sign).astype(np.uint16)
        vals = b.view(np.float16).astype(np.float32)
        for k in range(0, b.size, 97):            # a stride keeps this fast; end points added below
            v = float(vals[k])
            assert codec.h2f(int(b[k])) == v
            # -0.0 and +0.0 compare equal: accept either zero
            assert codec.h2f(codec.f2h_down(v)) == v
            assert codec.h2f(codec.f2h_up(v)) == v
    assert codec.h2f(codec.f2h_up(65504.0)) == 65504.0
    assert codec.h2f(codec.f2h_down(-65504.0)) == -65504.0


def test_half_directed_rounding_brackets_and_is_tight():
    rng = np.random.default_rng(1)
    xs = np.concatenate([rng.standard_normal(400) * 10.0 ** rng.integers(-7, 5, 400), [1e-9, -1e-9, 3e-8, 6.1e-5]])
    for x in xs.astype(np.float32):
        x = float(np.clip(x, -65504, 65504))
        lo = codec.h2f(codec.f2h_down(x))
        hi = codec.h2f(codec.f2h_up(x))
        assert lo <= x <= hi
        # tight: the bracket is one fp16 step wide at most (numpy's nextafter on float16 is the yardstick)
        if lo != hi:
            assert float(np.nextafter(np.float16(lo), np.float16(np.inf))) == hi
        # and agrees with round-to-nearest on one of the two ends
        assert float(np.float16(x)) in (lo, hi)


# ----------------------------------------------------------------------------- sub-fields and sizes

def test_subfields_are_binary_digits():
    expect = {0: [], 1: [(1, 0)], 2: [(2, 0)], 3: [(2, 1), (1, 0)], 4: [(4, 0)], 5: [(4, 1), (1, 0)],
              6: [(4, 2), (2, 0)], 7: [(4, 3), (2, 1), (1, 0)], 8: [(8, 0)]}
    for b, e in expect.items():
        got = codec.subfields(b)
        assert got == e
        assert sum(w for w, _ in got) == b
        # the sub-fields tile the code's bits exactly
        covered = sorted(itertools.chain.from_iterable(range(s, s + w) for w, s in got))
        assert covered == list(range(b))


@pytest.mark.parametrize("ratio,payload_bytes_per_token", [(4.0, 64), (8.0, 32), (12.0, 21.25)])
def test_packed_byte_count_matches_ratio_formula(ratio, payload_bytes_per_token):
    """Payload for N tokens is N * floor(16 d / ratio) / 8 bytes = N * 2 d / ratio for 4x and 8x against 16-bit
    elements; metadata adds 4 bytes per token per active scale group."""
    d, gs = 128, 64
    rng = np.random.default_rng(7)
    v = np.sort(rng.random(d) ** 4)[::-1] + 1e-9
    btot = fit.total_bits(d, ratio)
    widths = fit.alloc_bits(v, btot)
    assert widths.sum() == btot
    n_act = sum(widths[g * gs:(g + 1) * gs].any() for g in range(d // gs))
    tb = codec.tile_bytes(widths, gs)
    assert tb == 16 * btot + 512 * n_act
    assert (tb - 512 * n_act) / 128 == payload_bytes_per_token
    n_tokens = 32768
    assert (n_tokens // 128) * (tb - 512 * n_act) == n_tokens * btot // 8


# ----------------------------------------------------------------------------- layout: bijection and golden bytes

def _positions(widths, side):
    """(byte, bit) of every payload bit, gathered by packing one-hot codes through the packer."""
    d = widths.size
    gs = d
    tb = codec.tile_bytes(widths, gs)
    seen = {}
    for t in range(128):
        for j in range(d):
            for bit in range(int(widths[j])):
                tile = np.zeros(tb, np.uint8)
                codes = np.zeros(d, np.uint16)
                codes[j] = 1 << bit
                codec.pack_token(tile, widths, gs, side, t, codes, np.zeros(1, np.uint16), np.zeros(1, np.uint16))
                nz = np.nonzero(tile)[0]
                assert nz.size == 1
                byte = int(nz[0])
                v = int(tile[byte])
                assert v & (v - 1) == 0
                key = (byte, v.bit_length() - 1)
                assert key not in seen, "two code bits share a storage bit"
                seen[key] = (t, j, bit)
    return seen


@pytest.mark.parametrize("side", [codec.SIDE_K, codec.SIDE_V])
def test_layout_is_a_bijection_onto_the_payload(side):
    widths = np.array([7, 5, 3, 0, 1, 8, 2, 6], np.uint8)     # every sub-field class, odd and even strip counts
    seen = _positions(widths, side)
    payload_bits = 128 * int(widths.sum())
    assert len(seen) == payload_bits
    assert {b * 8 + k for b, k in seen} == set(range(payload_bits))


def _load_golden_bytes():
    out = {}
    with open(os.path.join(GOLDEN, "tile_layout_handworked.txt")) as f:
        for line in f:
            if line.startswith("byte "):
                _, ex, side, off, val = line.split()
                out.setdefault((ex, side), {})[int(off)] = int(val, 16)
    return out


def test_packer_reproduces_handworked_tiles():
    gold = _load_golden_bytes()
    wa = np.array([3, 1, 0, 2], np.uint8)
    toks = [(5, [5, 1, 0, 2], 0x3C00, 0x4000), (37, [7, 0, 0, 1], 0, 0), (53, [2, 1, 0, 3], 0, 0)]
    for side, name in ((codec.SIDE_K, "K"), (codec.SIDE_V, "V")):
        tile = np.zeros(codec.tile_bytes(wa, 4), np.uint8)
        assert tile.size == 608
        for t, c, lo, r in toks:
            codec.pack_token(tile, wa, 4, side, t, np.array(c, np.uint16), np.array([lo], np.uint16),
                             np.array([r], np.uint16))
        expect = np.zeros_like(tile)
        for off, val in gold[("A", name)].items():
            expect[off] = val
        assert np.array_equal(tile, expect)
    wb = np.array([1, 0, 0, 0], np.uint8)
    tile = np.zeros(codec.tile_bytes(wb, 4), np.uint8)
    assert tile.size == 528
    for t in (37, 127):
        codec.pack_token(tile, wb, 4, codec.SIDE_K, t, np.array([1, 0, 0, 0], np.uint16), np.zeros(1, np.uint16),
                         np.zeros(1, np.uint16))
    expect = np.zeros_like(tile)
    for off, val in gold[("B", "K")].items():
        expect[off] = val
    assert np.array_equal(tile, expect)


@pytest.mark.parametrize("side", [codec.SIDE_K, codec.SIDE_V])
def test_pack_unpack_every_code_every_width_every_slot(side):
    """Brute force: each width 1..8, each code value, at each token slot, written in scrambled order."""
    d, gs = 16, 8
    widths = np.array([1, 2, 3, 4, 5, 6, 7, 8, 8, 0, 3, 3, 1, 5, 0, 2], np.uint8)
    tb = codec.tile_bytes(widths, gs)
    rng = np.random.default_rng(3)
    for rep in range(3):
        tile = np.zeros(tb, np.uint8)
        codes = np.zeros((128, d), np.uint16)
        lo = rng.integers(0, 65536, (128, 2)).astype(np.uint16)
        r16 = rng.integers(0, 65536, (128, 2)).astype(np.uint16)
        for j in range(d):
            L = (1 << int(widths[j])) - 1
            # cycle through all values (plus noise) so every code value of every width appears
            codes[:, j] = (np.arange(128) * (rep + 1) + rng.integers(0, 256)) % (L + 1) if L else 0
        order = rng.permutation(128)
        for t in order:
            codec.pack_token(tile, widths, gs, side, int(t), codes[t], lo[t], r16[t])
        for t in range(128):
            c, l, r = codec.unpack_token(tile, widths, gs, side, t)
            assert np.array_equal(c, codes[t])
            assert np.array_equal(l, lo[t]) and np.array_equal(r, r16[t])
        # overwriting a slot replaces exactly that slot
        codec.pack_token(tile, widths, gs, side, 77, np.zeros(d, np.uint16), np.zeros(2, np.uint16),
                         np.zeros(2, np.uint16))
        c, _, _ = codec.unpack_token(tile, widths, gs, side, 77)
        assert not c.any()
        c, _, _ = codec.unpack_token(tile, widths, gs, side, 76)
        assert np.array_equal(c, codes[76])


def test_append_one_at_a_time_equals_bulk_encode():
    rng = np.random.default_rng(5)
    d, gs = 128, 64
    widths = fit.alloc_bits(np.arange(1, d + 1) ** -1.5, 512)
    y = rng.standard_normal((300, d)).astype(np.float32)
    tb = codec.tile_bytes(widths, gs)
    eye = np.eye(d, dtype=np.float32)
    zero = np.zeros(d, np.float32)
    for side in (codec.SIDE_K, codec.SIDE_V):
        bulk = np.zeros(3 * tb, np.uint8)
        codec.encode_unit(y, eye, zero, widths, gs, side, 0, bulk, tb, rotated_input=True)
        inc = np.zeros(3 * tb, np.uint8)
        for i in range(300):
            codec.encode_unit(y[i:i + 1], eye, zero, widths, gs, side, i, inc, tb, rotated_input=True)
        assert np.array_equal(bulk, inc)
        # slots of the tail tile that were never written stay zero
        c, l, r = codec.unpack_token(bulk[2 * tb:], widths, gs, side, 127)
        assert not c.any() and not l.any() and not r.any()


# ----------------------------------------------------------------------------- quantiser

def test_quantiser_range_extremes_and_error_bound():
    rng = np.random.default_rng(11)
    d, gs = 128, 64
    for trial in range(40):
        widths = rng.integers(0, 9, d).astype(np.uint8)
        y = (rng.standard_normal(d) * 10.0 ** rng.integers(-3, 3)).astype(np.float32)
        codes, lo16, r16, st = codec.quantise_token(y, widths, gs)
        assert st == 0
        yhat = codec.dequantise_token(codes, lo16, r16, widths, gs)
        for g in range(d // gs):
            sl = slice(g * gs, (g + 1) * gs)
            act = np.nonzero(widths[sl])[0] + g * gs
            if act.size == 0:
                assert lo16[g] == 0 and r16[g] == 0
                continue
            lo_f, r_f = codec.h2f(lo16[g]), codec.h2f(r16[g])
            # the stored range covers the data (directed rounding)
            assert lo_f <= y[act].min() and lo_f + r_f >= y[act].max()
            L = (1 << widths[act].astype(np.int64)) - 1
            assert (codes[act] <= L).all()
            assert codes[act[np.argmin(y[act])]] == 0
            assert codes[act[np.argmax(y[act])]] >= L[np.argmax(y[act])] - 1   # directed range may cost one level
            bound = r_f / (2.0 * L) * (1 + 1e-3) + 1e-30
            assert (np.abs(yhat[act].astype(np.float64) - y[act]) <= bound).all()
        assert (yhat[widths == 0] == 0).all() and (codes[widths == 0] == 0).all()


def test_quantiser_exact_range_hits_both_ends():
    # lo and hi exactly representable in fp16: the minimum maps to 0 and the maximum to L exactly
    widths = np.full(8, 4, np.uint8)
    y = np.array([-2.0, 6.0, 0.0, 1.0, 2.0, 3.0, 4.0, 5.5], np.float32)
    codes, lo16, r16, _ = codec.quantise_token(y, widths, 8)
    assert codec.h2f(lo16[0]) == -2.0 and codec.h2f(r16[0]) == 8.0
    assert codes[0] == 0 and codes[1] == 15
    # u = (y+2) * (15/8): y=0 -> 3.75 -> 4 ; y=2 -> 7.5 -> ties-to-even 8 ; y=-2+8/15*2.5.. skip
    assert codes[2] == 4 and codes[4] == 8
    yhat = codec.dequantise_token(codes, lo16, r16, widths, 8)
    assert yhat[0] == -2.0 and yhat[1] == 6.0


def test_quantiser_ties_round_to_even():
    # widths 2 -> L = 3, range [0, 3] -> inv = 1: u = y exactly; .5 cases must go to the even level
    widths = np.full(6, 2, np.uint8)
    y = np.array([0.0, 3.0, 0.5, 1.5, 2.5, 1.49999], np.float32)
    codes, _, _, _ = codec.quantise_token(y, widths, 6)
    assert list(codes) == [0, 3, 0, 2, 2, 1]


def test_quantiser_constant_group_and_single_channel():
    widths = np.array([3, 3, 0, 0, 5, 0, 0, 0], np.uint8)
    y = np.array([1.25, 1.25, 9.0, -9.0, 0.3, 100.0, 0, 0], np.float32)
    codes, lo16, r16, st = codec.quantise_token(y, widths, 4)
    assert st == 0
    # group 0: constant over its active channels (the zero-width channels do not widen the range)
    assert codec.h2f(lo16[0]) == 1.25 and codec.h2f(r16[0]) == 0.0 and codes[0] == 0 and codes[1] == 0
    yhat = codec.dequantise_token(codes, lo16, r16, widths, 4)
    assert yhat[0] == 1.25 and yhat[1] == 1.25 and yhat[2] == 0 and yhat[3] == 0
    # group 1: one active channel: range is rounded lo (down) and 0 or one fp16 step
    assert abs(yhat[4] - 0.3) <= 2.5e-4


def test_quantiser_flags_bad_inputs():
    widths = np.full(4, 4, np.uint8)
    _, _, _, st = codec.quantise_token(np.array([0, np.nan, 1, 2], np.float32), widths, 4)
    assert st & codec.STATUS_NONFINITE
    _, lo16, r16, st = codec.quantise_token(np.array([-1e6, 0, 1, 1e6], np.float32), widths, 4)
    assert st & codec.STATUS_F16_RANGE
    assert codec.h2f(lo16[0]) == -65504.0 and codec.h2f(r16[0]) == 65504.0


def test_sixteen_bit_budget_is_invertible_to_rounding():
    """At a 16-bit-equivalent budget the codec reproduces the rotated coordinates to 2^-16 of the group range."""
    rng = np.random.default_rng(13)
    d = 64
    widths = np.full(d, 16, np.uint8)
    y = rng.standard_normal(d).astype(np.float32) * 3
    codes, lo16, r16, _ = codec.quantise_token(y, widths, d)
    yhat = codec.dequantise_token(codes, lo16, r16, widths, d)
    r_f = codec.h2f(r16[0])
    assert np.abs(yhat.astype(np.float64) - y).max() <= r_f * 2.0 ** -16 * 0.5 * (1 + 1e-2) + 1e-7 * r_f
