"""Shared set-up for the GPU parity tests: draws a small workload, fits it with the oracle, and lays the same
parameters and caches out for both the oracle (numpy) and the CUDA library (torch device tensors)."""
import numpy as np

import spectra_inputs as si
from oracle import codec as oc
from oracle import fit as ofit


class Params:
    """Per-parameter-set transforms and widths for one side (numpy, the single source both sides read)."""

    def __init__(self, w_enc, w_dec, m_rot, widths, gs):
        self.w_enc = np.ascontiguousarray(w_enc, np.float32)     # [P, d, d]
        self.w_dec = np.ascontiguousarray(w_dec, np.float32)
        self.m_rot = np.ascontiguousarray(m_rot, np.float32)     # [P, d]
        self.widths = np.ascontiguousarray(widths, np.uint8)     # [P, d]
        self.gs = gs
        self.tile_bytes = np.array([oc.tile_bytes(w, gs) for w in self.widths], np.int64)

    @property
    def n_sets(self):
        return self.widths.shape[0]


def fit_params(xs_fit, ratio, gs=64, gain_mode=ofit.GAIN_SQRT, b_max=8, width_group=1, widths_override=None):
    """xs_fit: list of [n, d] arrays, one per parameter set."""
    we, wd, mr, ws = [], [], [], []
    for x in xs_fit:
        f = ofit.fit_basis(np.asarray(x, np.float64), gain_mode)
        we.append(f["W_enc"]); wd.append(f["W_dec"]); mr.append(f["m_rot"])
        if widths_override is not None:
            ws.append(np.asarray(widths_override, np.uint8))
        else:
            ws.append(ofit.alloc_bits(f["v_alloc"].astype(np.float32), ofit.total_bits(x.shape[1], ratio), b_max,
                                      width_group))
    return Params(np.stack(we), np.stack(wd), np.stack(mr), np.stack(ws), gs)


def cache_layout(params, n_units, cap_tokens):
    """Byte offsets of each unit-side's first tile for a capacity of cap_tokens tokens; total bytes."""
    cap_tiles = (cap_tokens + 127) // 128
    sizes = np.array([params.tile_bytes[u % params.n_sets] * cap_tiles for u in range(n_units)], np.int64)
    off = np.concatenate([[0], np.cumsum(sizes)[:-1]]).astype(np.int64)
    return off, int(sizes.sum())


def oracle_encode(params, side, x_units, pos0, cache, off, rotated=False):
    """x_units [n_units, n_new, d] float32.  Encodes into `cache` (numpy uint8) in place; returns status."""
    n_units = x_units.shape[0]
    st = 0
    for u in range(n_units):
        p = u % params.n_sets
        s, _ = oc.encode_unit(x_units[u], params.w_enc[p], params.m_rot[p], params.widths[p], params.gs, side,
                              int(pos0[u]), cache[off[u]:], int(params.tile_bytes[p]), rotated_input=rotated)
        st |= s
    return st


def unpack_codes(params, side, cache, off, u, n):
    p = u % params.n_sets
    tb = int(params.tile_bytes[p])
    codes = np.zeros((n, params.widths.shape[1]), np.uint16)
    metas = np.zeros((n, 2 * (params.widths.shape[1] // params.gs)), np.uint16)
    for t in range(n):
        c, lo, r = oc.unpack_token(cache[off[u] + (t // 128) * tb: off[u] + (t // 128 + 1) * tb], params.widths[p],
                                   params.gs, side, t % 128)
        codes[t] = c
        metas[t] = np.concatenate([lo, r])
    return codes, metas


def to_dev(a, device="cuda"):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def dev_params(params):
    return dict(w_enc=to_dev(params.w_enc), w_dec=to_dev(params.w_dec), m_rot=to_dev(params.m_rot),
                widths=to_dev(params.widths))


def rel_err_per_vector(got, ref):
    """max |got - ref| / max |ref| over the last axis, maximised over vectors."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    num = np.abs(got - ref).max(axis=-1)
    den = np.abs(ref).max(axis=-1)
    den = np.where(den > 0, den, 1.0)
    return float((num / den).max())


def draw_units(wl, layer, side, n_seq, n_tokens):
    """[n_seq * kv_heads, n_tokens, d] float32, units ordered [sequence][kv-head]."""
    out = np.zeros((n_seq * wl.kv_heads, n_tokens, wl.head_dim), np.float32)
    for s in range(n_seq):
        for h in range(wl.kv_heads):
            out[s * wl.kv_heads + h] = si.draw_unit(wl, layer, h, side, s, n_tokens=n_tokens)
    return out


def f16_ordinal(h):
    """Maps fp16 bit patterns to integers that are ordered like the values (adjacent values differ by one)."""
    h = np.asarray(h, np.uint16).astype(np.int32)
    return np.where(h & 0x8000, -(h & 0x7FFF), h & 0x7FFF)


def compare_coded_units(ref_cache, got_cache, tb, n, widths, gs, side):
    """Every token of one unit-side, the oracle's bytes against the library's: returns (entries that differ, active
    entries, largest code difference, largest metadata difference in fp16 steps, tokens whose metadata differ).
    Tokens whose metadata differ are not set apart: their entries count like all others."""
    cr, lr, rr = oc.unpack_unit(ref_cache, tb, n, widths, gs, side)
    cg, lg, rg = oc.unpack_unit(got_cache, tb, n, widths, gs, side)
    diff = np.abs(cr.astype(np.int32) - cg.astype(np.int32))
    active = int((np.asarray(widths) > 0).sum()) * n
    meta = np.maximum(np.abs(f16_ordinal(lr) - f16_ordinal(lg)), np.abs(f16_ordinal(rr) - f16_ordinal(rg)))
    return int((diff != 0).sum()), active, int(diff.max()), int(meta.max()), int((meta.max(axis=1) != 0).sum())
