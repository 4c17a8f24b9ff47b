"""Thin Python binding of libspectra (the C ABI declared in include/spectra.h).

Argument marshalling only: torch tensors supply device memory and the current CUDA stream; every
step of the codec runs in the library's CUDA kernels.  There is no fallback: if the shared
library is missing the first call raises.
"""
import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libspectra.so")
_lib = None

OK, INVALID_ARG, UNSUPPORTED, WORKSPACE_TOO_SMALL, CAPACITY, CUDA_ERROR = range(6)
F32, BF16 = 0, 1
SIDE_K, SIDE_V = 0, 1
ROTATED_INPUT = 1
STATUS_NONFINITE, STATUS_F16_RANGE, STATUS_WAIT_TIMEOUT, STATUS_CAPACITY, STATUS_BAD_LAYOUT = 1, 2, 4, 8, 16
PATH_CUDA_CORE, PATH_TENSOR_CORE = 0, 1
GAIN_ROTATE, GAIN_SQRT, GAIN_WHITEN = 0, 1, 2
HEAD_DIM = 128
TILE_TOKENS = 128
ATTENTION_LAUNCHES = 3   # kernels one spectra_decode_attention call enqueues
STEP_LAUNCHES = 3        # kernels one spectra_decode_step call enqueues on the tensor-core path (the append rides in the first)

EXPORTS = [
    "spectra_fit_basis", "spectra_fit_basis_static", "spectra_fit_workspace_bytes", "spectra_alloc_bits", "spectra_encode", "spectra_decode",
    "spectra_decode_attention", "spectra_decode_step", "spectra_attention_workspace_bytes", "spectra_tile_bytes", "spectra_config_default",
    "spectra_total_bits", "spectra_status_string", "spectra_cache_bytes", "spectra_attention_path",
    "spectra_alloc_bits_pooled", "spectra_split_ratio", "spectra_decode_rope", "spectra_decode_paged", "spectra_prefill_attention",
    "spectra_selftest_quotients",
]


class SpectraError(RuntimeError):
    pass


class Config(C.Structure):
    _fields_ = [("head_dim", C.c_int32), ("tile_tokens", C.c_int32), ("scale_group", C.c_int32),
                ("width_group", C.c_int32), ("b_max", C.c_int32), ("gain_mode", C.c_int32),
                ("layout_version", C.c_int32)]


def lib():
    """Loads libspectra.so; raises if it has not been built (no fallback path exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise SpectraError(f"{_LIB_PATH} is missing: build it with `python -m paper_2608_07915_b200.build`")
        _lib = C.CDLL(_LIB_PATH)
        _lib.spectra_fit_workspace_bytes.restype = C.c_size_t
        _lib.spectra_attention_workspace_bytes.restype = C.c_size_t
        _lib.spectra_tile_bytes.restype = C.c_size_t
        _lib.spectra_cache_bytes.restype = C.c_size_t
        _lib.spectra_total_bits.restype = C.c_int32
        _lib.spectra_status_string.restype = C.c_char_p
        _lib.spectra_config_default.restype = None
    return _lib


def default_config(**overrides):
    cfg = Config()
    lib().spectra_config_default(C.byref(cfg))
    for k, v in overrides.items():
        setattr(cfg, k, int(v))
    return cfg


def status_string(code):
    return lib().spectra_status_string(C.c_int(code)).decode()


def selftest_quotients(mismatches):
    """mismatches: int64 device tensor of one element; receives how many quotients (2^b - 1) / R16 of the bulk
    encoder differ from the IEEE division over every positive finite fp16 R16 and b = 1..8 (0 is the only
    acceptable answer).  Runs on the current stream."""
    _check(lib().spectra_selftest_quotients(_ptr(mismatches), _stream()), "spectra_selftest_quotients")


def _check(rc, what):
    if rc != OK:
        raise SpectraError(f"{what}: {status_string(rc)}")


def _ptr(t):
    return C.c_void_p(0 if t is None else t.data_ptr())


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dtype_code(t):
    import torch
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise SpectraError(f"unsupported tensor dtype {t.dtype}")


def cache_bytes(cfg, widths_host, capacity_tokens):
    """Bytes of one unit-side's buffer that holds capacity_tokens tokens (whole tiles)."""
    arr = (C.c_uint8 * HEAD_DIM)(*[int(w) for w in widths_host])
    return int(lib().spectra_cache_bytes(C.byref(cfg), arr, C.c_int64(capacity_tokens)))


def attention_path(cfg, n_kv_heads, n_q_heads, n_param_sets, widths_k_host, widths_v_host):
    """PATH_TENSOR_CORE or PATH_CUDA_CORE: the kernels decode_attention / decode_step will run for these host widths
    (numpy uint8 [n_param_sets, 128] each, or None)."""
    wk = wv = C.c_void_p(0)
    if widths_k_host is not None and widths_v_host is not None:
        assert widths_k_host.dtype.name == "uint8" and widths_k_host.flags.c_contiguous
        assert widths_v_host.dtype.name == "uint8" and widths_v_host.flags.c_contiguous
        wk = widths_k_host.ctypes.data_as(C.c_void_p)
        wv = widths_v_host.ctypes.data_as(C.c_void_p)
    rc = int(lib().spectra_attention_path(C.byref(cfg), C.c_int32(n_kv_heads), C.c_int32(n_q_heads),
                                          C.c_int64(n_param_sets), wk, wv))
    if rc < 0:
        raise SpectraError("spectra_attention_path: invalid arguments")
    return rc


def tile_bytes(cfg, widths_host):
    """widths_host: 128 integers (any sequence).  Bytes of one packed tile."""
    arr = (C.c_uint8 * HEAD_DIM)(*[int(w) for w in widths_host])
    n = lib().spectra_tile_bytes(C.byref(cfg), arr)
    if n == 0 and any(int(w) for w in widths_host):
        raise SpectraError("spectra_tile_bytes: bad arguments")
    return int(n)


def total_bits(cfg, ratio):
    return int(lib().spectra_total_bits(C.byref(cfg), C.c_double(ratio)))


def fit_workspace_bytes(cfg, n_units):
    return int(lib().spectra_fit_workspace_bytes(C.byref(cfg), C.c_int64(n_units)))


def attention_workspace_bytes(cfg, batch, n_kv_heads, n_q_heads, max_seq_len):
    return int(lib().spectra_attention_workspace_bytes(C.byref(cfg), C.c_int32(batch), C.c_int32(n_kv_heads),
                                                       C.c_int32(n_q_heads), C.c_int32(max_seq_len)))


def fit_basis(cfg, x, n_units, n_tokens, stride_unit, stride_token, w_enc, w_dec, mean_rot, var_alloc,
              eigval=None, basis_u=None, workspace=None):
    rc = lib().spectra_fit_basis(C.byref(cfg), _ptr(x), C.c_int(_dtype_code(x)), C.c_int64(n_units),
                                 C.c_int64(n_tokens), C.c_int64(stride_unit), C.c_int64(stride_token), _ptr(w_enc),
                                 _ptr(w_dec), _ptr(mean_rot), _ptr(var_alloc), _ptr(eigval), _ptr(basis_u),
                                 _ptr(workspace), C.c_size_t(0 if workspace is None else workspace.numel() *
                                                             workspace.element_size()), _stream())
    _check(rc, "spectra_fit_basis")


FIT_STATIC_MAX_UNITS = 8


def fit_basis_static(cfg, x, n_units, n_tokens, stride_unit, stride_token, w_enc, w_dec, mean_rot, var_alloc,
                     eigval=None, basis_u=None):
    """spectra_fit_basis without a workspace argument, for callers that cannot allocate device memory when they
    calibrate: the scratch is a fixed array inside the library (at most FIT_STATIC_MAX_UNITS unit-sides per call).
    Make the first call on a device outside stream capture; do not overlap two calls on one device."""
    rc = lib().spectra_fit_basis_static(C.byref(cfg), _ptr(x), C.c_int(_dtype_code(x)), C.c_int64(n_units),
                                        C.c_int64(n_tokens), C.c_int64(stride_unit), C.c_int64(stride_token),
                                        _ptr(w_enc), _ptr(w_dec), _ptr(mean_rot), _ptr(var_alloc), _ptr(eigval),
                                        _ptr(basis_u), _stream())
    _check(rc, "spectra_fit_basis_static")


def alloc_bits(cfg, var_alloc, n_units, ratio, widths):
    rc = lib().spectra_alloc_bits(C.byref(cfg), _ptr(var_alloc), C.c_int64(n_units), C.c_double(ratio), _ptr(widths),
                                  _stream())
    _check(rc, "spectra_alloc_bits")


def alloc_bits_pooled(cfg, var_alloc, n_units, pool_units, ratio, widths):
    """Allocation with the budget pooled over runs of pool_units consecutive units (the heads of a layer)."""
    rc = lib().spectra_alloc_bits_pooled(C.byref(cfg), _ptr(var_alloc), C.c_int64(n_units), C.c_int64(pool_units),
                                         C.c_double(ratio), _ptr(widths), _stream())
    _check(rc, "spectra_alloc_bits_pooled")


def split_ratio(ratio, kappa):
    """(ratio_k, ratio_v): the keys get the fraction kappa of the bits of keys and values together."""
    rk, rv = C.c_double(0), C.c_double(0)
    _check(lib().spectra_split_ratio(C.c_double(ratio), C.c_double(kappa), C.byref(rk), C.byref(rv)),
           "spectra_split_ratio")
    return rk.value, rv.value


def encode(cfg, side, x, flags, n_units, n_param_sets, pos0, n_new, stride_unit, stride_token, w_enc, mean_rot,
           widths, cache, unit_offset, status_word=None, capacity_tokens=0, tile_table=None, table_stride=0):
    """capacity_tokens: tokens each unit-side's buffer holds (0: not checked).  tile_table: device int32
    [n_units, table_stride] page indices of a paged cache (None: contiguous tiles)."""
    rc = lib().spectra_encode(C.byref(cfg), C.c_int(side), _ptr(x), C.c_int(_dtype_code(x)), C.c_int(flags),
                              C.c_int64(n_units), C.c_int64(n_param_sets), _ptr(pos0), C.c_int32(n_new),
                              C.c_int64(stride_unit), C.c_int64(stride_token), _ptr(w_enc), _ptr(mean_rot),
                              _ptr(widths), _ptr(cache), _ptr(unit_offset), C.c_int32(capacity_tokens),
                              _ptr(tile_table), C.c_int64(table_stride), _ptr(status_word), _stream())
    _check(rc, "spectra_encode")


def decode(cfg, side, cache, unit_offset, n_units, n_param_sets, n_tokens, max_tokens, w_dec, mean_rot, widths, out,
           yhat_out, stride_unit, stride_token, status_word=None, tile_table=None, table_stride=0):
    out_code = _dtype_code(out) if out is not None else F32
    rc = lib().spectra_decode(C.byref(cfg), C.c_int(side), _ptr(cache), _ptr(unit_offset), C.c_int64(n_units),
                              C.c_int64(n_param_sets), _ptr(n_tokens), C.c_int32(max_tokens), _ptr(w_dec),
                              _ptr(mean_rot), _ptr(widths), _ptr(out), C.c_int(out_code), _ptr(yhat_out),
                              C.c_int64(stride_unit), C.c_int64(stride_token), _ptr(tile_table), C.c_int64(table_stride),
                              _ptr(status_word), _stream())
    _check(rc, "spectra_decode")


def decode_rope(cfg, cache, unit_offset, n_units, n_param_sets, n_tokens, max_tokens, w_dec, mean_rot, widths, out,
                stride_unit, stride_token, rope_cos, rope_sin, position0=None, status_word=None, tile_table=None,
                table_stride=0):
    """Reconstructs keys and applies the rotary position embedding (rotate-half pairing) from cos / sin tables
    [positions, 64]; position0: device int32 [n_units] (None: 0)."""
    rc = lib().spectra_decode_rope(C.byref(cfg), _ptr(cache), _ptr(unit_offset), C.c_int64(n_units),
                                   C.c_int64(n_param_sets), _ptr(n_tokens), C.c_int32(max_tokens), _ptr(w_dec),
                                   _ptr(mean_rot), _ptr(widths), _ptr(out), C.c_int(_dtype_code(out)),
                                   C.c_int64(stride_unit), C.c_int64(stride_token), _ptr(tile_table),
                                   C.c_int64(table_stride), _ptr(position0), _ptr(rope_cos), _ptr(rope_sin),
                                   _ptr(status_word), _stream())
    _check(rc, "spectra_decode_rope")


def decode_paged(cfg, side, cache, unit_offset, n_units, n_param_sets, n_tokens, max_tokens, w_dec, mean_rot, widths,
                 out_pool, stride_page, stride_token, out_table, out_table_stride, tile_table=None, table_stride=0,
                 position0=None, rope_cos=None, rope_sin=None, status_word=None):
    """Reconstruction into a pool of 128-token pages: tile t of unit u goes to page out_table[u, t] (device int32)."""
    rc = lib().spectra_decode_paged(C.byref(cfg), C.c_int(side), _ptr(cache), _ptr(unit_offset), C.c_int64(n_units),
                                    C.c_int64(n_param_sets), _ptr(n_tokens), C.c_int32(max_tokens), _ptr(w_dec),
                                    _ptr(mean_rot), _ptr(widths), _ptr(out_pool), C.c_int(_dtype_code(out_pool)),
                                    C.c_int64(stride_page), C.c_int64(stride_token), _ptr(tile_table),
                                    C.c_int64(table_stride), _ptr(out_table), C.c_int64(out_table_stride),
                                    _ptr(position0), _ptr(rope_cos), _ptr(rope_sin), _ptr(status_word), _stream())
    _check(rc, "spectra_decode_paged")


def prefill_attention(q, k_pool, v_pool, n_pages, stride_page, stride_token, page_table, table_stride, n_seqs,
                      n_kv_heads, n_q_heads, pos0, n_new, q_strides, softmax_scale, out, out_strides, lse=None,
                      status_word=None):
    """Causal attention of n_new queries per sequence over reconstructed bf16 page pools.  q_strides, out_strides:
    (sequence, token, head) strides in elements."""
    rc = lib().spectra_prefill_attention(_ptr(q), _ptr(k_pool), _ptr(v_pool), C.c_int64(n_pages),
                                         C.c_int64(stride_page), C.c_int64(stride_token), _ptr(page_table),
                                         C.c_int64(table_stride), C.c_int64(n_seqs), C.c_int32(n_kv_heads),
                                         C.c_int32(n_q_heads), _ptr(pos0), C.c_int32(n_new), C.c_int64(q_strides[0]),
                                         C.c_int64(q_strides[1]), C.c_int64(q_strides[2]), C.c_float(softmax_scale),
                                         _ptr(out), C.c_int64(out_strides[0]), C.c_int64(out_strides[1]),
                                         C.c_int64(out_strides[2]), _ptr(lse), _ptr(status_word), _stream())
    _check(rc, "spectra_prefill_attention")


def decode_attention(cfg, q, batch, n_kv_heads, n_q_heads, seq_len, max_seq_len, cache_k, unit_offset_k, cache_v,
                     unit_offset_v, n_param_sets, w_dec_k, mean_rot_k, widths_k, w_dec_v, mean_rot_v, widths_v,
                     softmax_scale, out, lse, workspace, status_word=None, widths_k_host=None, widths_v_host=None,
                     tile_table_k=None, tile_table_v=None, table_stride=0):
    """widths_*_host: optional numpy uint8 arrays [n_param_sets, 128] (host copies of the widths); they select the
    tensor-core kernel.  tile_table_*: device int32 [n_units, table_stride] page indices of paged caches."""
    wkh = wvh = C.c_void_p(0)
    if widths_k_host is not None:
        assert widths_k_host.dtype.name == "uint8" and widths_k_host.flags.c_contiguous
        assert widths_v_host.dtype.name == "uint8" and widths_v_host.flags.c_contiguous
        assert widths_k_host.size == n_param_sets * HEAD_DIM == widths_v_host.size
        wkh = widths_k_host.ctypes.data_as(C.c_void_p)
        wvh = widths_v_host.ctypes.data_as(C.c_void_p)
    rc = lib().spectra_decode_attention(
        C.byref(cfg), _ptr(q), C.c_int(_dtype_code(q)), C.c_int32(batch), C.c_int32(n_kv_heads), C.c_int32(n_q_heads),
        _ptr(seq_len), C.c_int32(max_seq_len), _ptr(cache_k), _ptr(unit_offset_k), _ptr(cache_v),
        _ptr(unit_offset_v), C.c_int64(n_param_sets), _ptr(w_dec_k), _ptr(mean_rot_k), _ptr(widths_k), _ptr(w_dec_v),
        _ptr(mean_rot_v), _ptr(widths_v), wkh, wvh, C.c_float(softmax_scale), _ptr(out), C.c_int(_dtype_code(out)), _ptr(lse),
        _ptr(workspace), C.c_size_t(workspace.numel() * workspace.element_size()), _ptr(tile_table_k),
        _ptr(tile_table_v), C.c_int64(table_stride), _ptr(status_word), _stream())
    _check(rc, "spectra_decode_attention")


def decode_step(cfg, q, new_k, new_v, batch, n_kv_heads, n_q_heads, seq_len, max_seq_len, cache_k, unit_offset_k,
                cache_v, unit_offset_v, n_param_sets, w_enc_k, w_dec_k, mean_rot_k, widths_k, w_enc_v, w_dec_v,
                mean_rot_v, widths_v, softmax_scale, out, lse, workspace, status_word=None, widths_k_host=None,
                widths_v_host=None, tile_table_k=None, tile_table_v=None, table_stride=0):
    """One decode step of a layer: appends new_k / new_v ([batch * n_kv_heads, 128], one vector per unit) at
    position seq_len - 1 and attends over seq_len tokens (seq_len already counts the new token)."""
    wkh = wvh = C.c_void_p(0)
    if widths_k_host is not None:
        assert widths_k_host.dtype.name == "uint8" and widths_k_host.flags.c_contiguous
        assert widths_v_host.dtype.name == "uint8" and widths_v_host.flags.c_contiguous
        assert widths_k_host.size == n_param_sets * HEAD_DIM == widths_v_host.size
        wkh = widths_k_host.ctypes.data_as(C.c_void_p)
        wvh = widths_v_host.ctypes.data_as(C.c_void_p)
    assert new_k.dtype == new_v.dtype and new_k.is_contiguous() and new_v.is_contiguous()
    rc = lib().spectra_decode_step(
        C.byref(cfg), _ptr(q), C.c_int(_dtype_code(q)), _ptr(new_k), _ptr(new_v), C.c_int(_dtype_code(new_k)),
        C.c_int32(batch), C.c_int32(n_kv_heads), C.c_int32(n_q_heads), _ptr(seq_len), C.c_int32(max_seq_len),
        _ptr(cache_k), _ptr(unit_offset_k), _ptr(cache_v), _ptr(unit_offset_v), C.c_int64(n_param_sets),
        _ptr(w_enc_k), _ptr(w_dec_k), _ptr(mean_rot_k), _ptr(widths_k), _ptr(w_enc_v), _ptr(w_dec_v), _ptr(mean_rot_v),
        _ptr(widths_v), wkh, wvh, C.c_float(softmax_scale), _ptr(out), C.c_int(_dtype_code(out)), _ptr(lse),
        _ptr(workspace), C.c_size_t(workspace.numel() * workspace.element_size()), _ptr(tile_table_k),
        _ptr(tile_table_v), C.c_int64(table_stride), _ptr(status_word), _stream())
    _check(rc, "spectra_decode_step")
