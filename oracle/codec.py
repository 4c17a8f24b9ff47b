"""CPU oracle (test infrastructure): ctypes front end of spectra_oracle.c.

Argument marshalling only; every arithmetic step is in the C file.  The shared object is built
by `build()` with gcc (-O2 -ffp-contract=off; OpenMP over independent units only).
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spectra_oracle.c")
_SO = os.path.join(_HERE, "libspectra_oracle.so")
_lib = None

SIDE_K, SIDE_V = 0, 1
TILE = 128
STATUS_NONFINITE, STATUS_F16_RANGE = 1, 2


def build(force=False):
    if not force and os.path.exists(_SO) and os.path.getmtime(_SO) >= os.path.getmtime(_SRC):
        return _SO
    cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC", "-o", _SO, _SRC,
           "-lm"]
    subprocess.check_call(cmd)
    return _SO


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_SO)
        _lib.spo_tile_bytes.restype = C.c_int64
        _lib.spo_h2f.restype = C.c_float
        _lib.spo_f2h_down.restype = C.c_uint16
        _lib.spo_f2h_up.restype = C.c_uint16
        _lib.spo_f2h_down.argtypes = [C.c_float]
        _lib.spo_f2h_up.argtypes = [C.c_float]
        _lib.spo_h2f.argtypes = [C.c_uint16]
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _u8(a):
    return np.ascontiguousarray(a, dtype=np.uint8)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def num_threads():
    return int(lib().spo_num_threads())


def set_num_threads(n):
    lib().spo_set_num_threads(C.c_int(int(n)))


def f2h_down(x):
    return int(lib().spo_f2h_down(C.c_float(float(x))))


def f2h_up(x):
    return int(lib().spo_f2h_up(C.c_float(float(x))))


def h2f(h):
    return float(lib().spo_h2f(C.c_uint16(int(h))))


def subfields(b):
    w = (C.c_int * 4)()
    s = (C.c_int * 4)()
    n = lib().spo_subfields(C.c_int(int(b)), w, s)
    return [(int(w[i]), int(s[i])) for i in range(n)]


def tile_bytes(widths, gs):
    widths = _u8(widths)
    return int(lib().spo_tile_bytes(_p(widths), C.c_int(widths.size), C.c_int(gs)))


def strip_table(widths, side):
    widths = _u8(widths)
    d = widths.size
    chan = np.zeros(3 * d, np.int32)
    w = np.zeros(3 * d, np.int32)
    shift = np.zeros(3 * d, np.int32)
    mode = np.zeros(3 * d, np.int32)
    base = np.zeros(3 * d, np.int64)
    n = lib().spo_strip_table(_p(widths), C.c_int(d), C.c_int(side), _p(chan), _p(w), _p(shift), _p(mode), _p(base))
    return dict(chan=chan[:n], w=w[:n], shift=shift[:n], mode=mode[:n], base=base[:n])


def quantise_token(y, widths, gs):
    y = _f32(y)
    widths = _u8(widths)
    d = y.size
    codes = np.zeros(d, np.uint16)
    lo16 = np.zeros(d // gs, np.uint16)
    r16 = np.zeros(d // gs, np.uint16)
    st = lib().spo_quantise_token(_p(y), _p(widths), C.c_int(d), C.c_int(gs), _p(codes), _p(lo16), _p(r16))
    return codes, lo16, r16, int(st)


def dequantise_token(codes, lo16, r16, widths, gs):
    codes = np.ascontiguousarray(codes, np.uint16)
    lo16 = np.ascontiguousarray(lo16, np.uint16)
    r16 = np.ascontiguousarray(r16, np.uint16)
    widths = _u8(widths)
    d = codes.size
    out = np.zeros(d, np.float32)
    lib().spo_dequantise_token(_p(codes), _p(lo16), _p(r16), _p(widths), C.c_int(d), C.c_int(gs), _p(out))
    return out


def pack_token(tile, widths, gs, side, t, codes, lo16, r16):
    widths = _u8(widths)
    assert tile.dtype == np.uint8 and tile.flags.c_contiguous
    codes = np.ascontiguousarray(codes, np.uint16)
    lo16 = np.ascontiguousarray(lo16, np.uint16)
    r16 = np.ascontiguousarray(r16, np.uint16)
    lib().spo_pack_token(_p(tile), _p(widths), C.c_int(widths.size), C.c_int(gs), C.c_int(side), C.c_int(t),
                         _p(codes), _p(lo16), _p(r16))


def unpack_token(tile, widths, gs, side, t):
    widths = _u8(widths)
    d = widths.size
    codes = np.zeros(d, np.uint16)
    lo16 = np.zeros(d // gs, np.uint16)
    r16 = np.zeros(d // gs, np.uint16)
    tile = _u8(tile)
    lib().spo_unpack_token(_p(tile), _p(widths), C.c_int(d), C.c_int(gs), C.c_int(side), C.c_int(t), _p(codes),
                           _p(lo16), _p(r16))
    return codes, lo16, r16


def unpack_unit(cache, tile_stride, n, widths, gs, side):
    """Codes [n, d] and metadata lo16, R16 [n, d / gs] of tokens [0, n) of one unit-side (cache starts at its
    first tile)."""
    widths = _u8(widths)
    d = widths.size
    cache = _u8(cache)
    codes = np.zeros((n, d), np.uint16)
    lo16 = np.zeros((n, d // gs), np.uint16)
    r16 = np.zeros((n, d // gs), np.uint16)
    lib().spo_unpack_unit(_p(cache), C.c_int64(tile_stride), C.c_int64(n), _p(widths), C.c_int(d), C.c_int(gs),
                          C.c_int(side), _p(codes), _p(lo16), _p(r16))
    return codes, lo16, r16


def rotate_token(x, w_enc, m_rot):
    x = _f32(x)
    w_enc = _f32(w_enc)
    m_rot = _f32(m_rot)
    y = np.zeros(x.size, np.float32)
    lib().spo_rotate_token(_p(x), _p(w_enc), _p(m_rot), C.c_int(x.size), _p(y))
    return y


def encode_unit(x, w_enc, m_rot, widths, gs, side, pos0, cache, tile_stride, rotated_input=False, want_codes=False):
    """Append the rows of x ([n_new, d] float32) at positions pos0.. into `cache` (uint8 array that starts at
    the unit-side's first tile).  Returns (status, codes or None)."""
    x = _f32(x)
    n_new, d = x.shape
    w_enc = _f32(w_enc)
    m_rot = _f32(m_rot)
    widths = _u8(widths)
    assert cache.dtype == np.uint8 and cache.flags.c_contiguous
    codes = np.zeros((n_new, d), np.uint16) if want_codes else None
    st = lib().spo_encode_unit(_p(x), C.c_int(int(rotated_input)), _p(w_enc), _p(m_rot), _p(widths), C.c_int(d),
                               C.c_int(gs), C.c_int(side), C.c_int64(pos0), C.c_int64(n_new), _p(cache),
                               C.c_int64(tile_stride), _p(codes) if want_codes else None)
    return int(st), codes


def decode_unit(cache, tile_stride, n, w_dec, m_rot, widths, gs, side, want_yhat=True, want_xhat=True):
    cache = _u8(cache)
    w_dec = _f32(w_dec)
    m_rot = _f32(m_rot)
    widths = _u8(widths)
    d = widths.size
    yhat = np.zeros((n, d), np.float32) if want_yhat else None
    xhat = np.zeros((n, d), np.float64) if want_xhat else None
    lib().spo_decode_unit(_p(cache), C.c_int64(tile_stride), C.c_int64(n), _p(w_dec), _p(m_rot), _p(widths),
                          C.c_int(d), C.c_int(gs), C.c_int(side), _p(yhat) if want_yhat else None,
                          _p(xhat) if want_xhat else None)
    return yhat, xhat


def attention_units(mode, q, n_tokens, cache_k, off_k, stride_k, cache_v, off_v, stride_v, w_dec_k, m_rot_k,
                    widths_k, w_dec_v, m_rot_v, widths_v, gs, scale):
    """mode 'A' (reconstruct then attend) or 'B' (latent-space).  q [n_units, G, d].  Returns out, lse (fp64)."""
    q = _f64(q)
    n_units, G, d = q.shape
    out = np.zeros((n_units, G, d), np.float64)
    lse = np.zeros((n_units, G), np.float64)
    args = [_i64(n_tokens), _u8(cache_k), _i64(off_k), _i64(stride_k), _u8(cache_v), _i64(off_v), _i64(stride_v),
            _f32(w_dec_k), _f32(m_rot_k), _u8(widths_k), _f32(w_dec_v), _f32(m_rot_v), _u8(widths_v)]
    lib().spo_attention_units(C.c_int(0 if mode == "A" else 1), _p(q), C.c_int(G), C.c_int64(n_units), _p(args[0]),
                              _p(args[1]), _p(args[2]), _p(args[3]), _p(args[4]), _p(args[5]), _p(args[6]),
                              _p(args[7]), _p(args[8]), _p(args[9]), _p(args[10]), _p(args[11]), _p(args[12]),
                              C.c_int(d), C.c_int(gs), C.c_double(scale), _p(out), _p(lse))
    return out, lse


def encode_units(x, w_enc, m_rot, widths, gs, side, pos0, cache, unit_offset, tile_stride, rotated_input=False):
    """x [n_units, n_new, d] float32; per-unit w_enc [n_units, d, d], m_rot, widths [n_units, d]."""
    x = _f32(x)
    n_units, n_new, d = x.shape
    st = lib().spo_encode_units(_p(x), C.c_int64(n_new * d), C.c_int(int(rotated_input)), _p(_f32(w_enc)),
                                _p(_f32(m_rot)), _p(_u8(widths)), C.c_int(d), C.c_int(gs), C.c_int(side),
                                C.c_int64(n_units), C.c_int64(pos0), C.c_int64(n_new), _p(cache),
                                _p(_i64(unit_offset)), _p(_i64(tile_stride)))
    return int(st)


def rope_rows(x, pos0, theta):
    """Rotates row t of x ([n, d] fp64) at position pos0 + t (rotate-half pairing).  Returns a new array."""
    x = _f64(x).copy()
    n, d = x.shape
    for t in range(n):
        lib().spo_rope_row(_p(x[t]), C.c_int(d), C.c_double(pos0 + t), C.c_double(theta))
    return x


def decode_unit_rope(cache, tile_stride, n, w_dec, m_rot, widths, gs, side, pos0, theta):
    cache = _u8(cache)
    widths = _u8(widths)
    d = widths.size
    xhat = np.zeros((n, d), np.float64)
    lib().spo_decode_unit_rope(_p(cache), C.c_int64(tile_stride), C.c_int64(n), _p(_f32(w_dec)), _p(_f32(m_rot)),
                               _p(widths), C.c_int(d), C.c_int(gs), C.c_int(side), C.c_double(pos0), C.c_double(theta),
                               _p(xhat))
    return xhat


def attention_rope_unit(mode, q, n, cache_k, stride_k, cache_v, stride_v, w_dec_k, m_rot_k, widths_k, w_dec_v, m_rot_v,
                        widths_v, gs, scale, pos0, theta):
    """One unit, q [G, d] (already rotated at the query's position).  mode 'A' or 'B'.  Returns out [G, d], lse [G]."""
    q = _f64(q)
    G, d = q.shape
    out = np.zeros((G, d), np.float64)
    lse = np.zeros(G, np.float64)
    fn = lib().spo_attention_rope_mode_a if mode == "A" else lib().spo_attention_rope_mode_b
    fn(_p(q), C.c_int(G), _p(_u8(cache_k)), C.c_int64(stride_k), _p(_u8(cache_v)), C.c_int64(stride_v), C.c_int64(n),
       _p(_f32(w_dec_k)), _p(_f32(m_rot_k)), _p(_u8(widths_k)), _p(_f32(w_dec_v)), _p(_f32(m_rot_v)), _p(_u8(widths_v)),
       C.c_int(d), C.c_int(gs), C.c_double(scale), C.c_double(pos0), C.c_double(theta), _p(out), _p(lse))
    return out, lse
