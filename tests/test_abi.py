"""The C-ABI library loads, exports every symbol the header declares, and rejects bad arguments on the host
(no GPU needed: argument validation happens before any CUDA call)."""
import ctypes as C
import os
import re

import pytest

import paper_2608_07915_b200 as sp
from paper_2608_07915_b200 import build as sp_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    sp_build.build()
    return sp.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "spectra.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spectra_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert "spectra_decode_attention" in names and "spectra_fit_basis" in names and len(names) >= 11
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(sp.EXPORTS) == names


def test_config_default_and_host_helpers(lib):
    cfg = sp.default_config()
    assert (cfg.head_dim, cfg.tile_tokens, cfg.scale_group, cfg.width_group, cfg.b_max, cfg.layout_version) == \
        (128, 128, 64, 1, 8, 1)
    assert sp.total_bits(cfg, 4.0) == 512 and sp.total_bits(cfg, 8.0) == 256 and sp.total_bits(cfg, 12.0) == 170
    assert sp.total_bits(cfg, 1.0) == 1024                      # clamped to b_max * d
    w = [4] * 128
    assert sp.tile_bytes(cfg, w) == 16 * 512 + 1024              # 9216 bytes: 3.56x against 32768
    assert sp.tile_bytes(cfg, [2] * 64 + [0] * 64) == 16 * 128 + 512
    assert sp.tile_bytes(cfg, [0] * 128) == 0
    assert sp.status_string(0) == "SPECTRA_OK" and sp.status_string(3) == "SPECTRA_WORKSPACE_TOO_SMALL"
    assert sp.fit_workspace_bytes(cfg, 2) >= 2 * (128 * 128 + 128) * 8
    assert sp.attention_workspace_bytes(cfg, 8, 8, 32, 32768) > 0


def test_bad_arguments_are_rejected_before_any_launch(lib):
    cfg = sp.default_config()
    null = C.c_void_p(0)
    bad = sp.default_config(head_dim=64)
    assert lib.spectra_alloc_bits(C.byref(bad), null, C.c_int64(1), C.c_double(4.0), null, null) == sp.UNSUPPORTED
    assert lib.spectra_alloc_bits(C.byref(cfg), null, C.c_int64(1), C.c_double(4.0), null, null) == sp.INVALID_ARG
    assert lib.spectra_alloc_bits(C.byref(cfg), null, C.c_int64(0), C.c_double(4.0), null, null) == sp.OK
    assert lib.spectra_alloc_bits(C.byref(cfg), null, C.c_int64(1), C.c_double(-1.0), null, null) == sp.INVALID_ARG
    assert lib.spectra_alloc_bits(None, null, C.c_int64(1), C.c_double(4.0), null, null) == sp.INVALID_ARG
    bad = sp.default_config(scale_group=48)
    assert lib.spectra_fit_workspace_bytes(C.byref(bad), C.c_int64(1)) == 0
    bad = sp.default_config(b_max=9)
    assert lib.spectra_encode(C.byref(bad), 0, null, 0, 0, C.c_int64(1), C.c_int64(1), null, 1, C.c_int64(0),
                              C.c_int64(0), null, null, null, null, null, 0, null, C.c_int64(0), null,
                              null) == sp.INVALID_ARG
    # rotated input must be fp32; unknown flags; bad side
    args = (C.c_int64(1), C.c_int64(1), null, 1, C.c_int64(0), C.c_int64(0), null, null, null, null, null, 0, null,
            C.c_int64(0), null, null)
    assert lib.spectra_encode(C.byref(cfg), 0, null, sp.BF16, sp.ROTATED_INPUT, *args) == sp.INVALID_ARG
    assert lib.spectra_encode(C.byref(cfg), 0, null, sp.F32, 8, *args) == sp.INVALID_ARG
    assert lib.spectra_encode(C.byref(cfg), 2, null, sp.F32, 0, *args) == sp.INVALID_ARG
    assert lib.spectra_encode(C.byref(cfg), 0, null, sp.F32, 0, *args) == sp.INVALID_ARG     # null pointers
    neg = (C.c_int64(1), C.c_int64(1), null, 1, C.c_int64(0), C.c_int64(0), null, null, null, null, null, -5, null,
           C.c_int64(0), null, null)
    assert lib.spectra_encode(C.byref(cfg), 0, null, sp.F32, 0, *neg) == sp.INVALID_ARG      # negative capacity
    # attention: query heads must be a multiple of kv heads; group size above 8 unsupported
    def attn(n_kv, n_q):
        return lib.spectra_decode_attention(C.byref(cfg), null, 0, 1, n_kv, n_q, null, 128, null, null, null, null,
                                            C.c_int64(1), null, null, null, null, null, null, C.c_float(0), null, 0,
                                            null, null, C.c_size_t(0), null, null, C.c_int64(0), null, null)
    assert attn(3, 8) == sp.INVALID_ARG
    assert attn(1, 16) == sp.UNSUPPORTED
    assert attn(2, 8) == sp.INVALID_ARG                                                      # null pointers


def test_misaligned_buffers_are_refused_on_the_host(lib):
    """The kernels use 16-byte (attention, encode) and 2-byte (decode) accesses on these buffers; the entry points
    check the alignment before anything is launched (the pointers below are never dereferenced)."""
    cfg = sp.default_config()
    null = C.c_void_p(0)
    p = lambda a: C.c_void_p(a)
    ok = 0x10000
    # spectra_encode: cache one byte off
    assert lib.spectra_encode(C.byref(cfg), 0, p(ok), sp.F32, 0, C.c_int64(1), C.c_int64(1), p(ok), 1, C.c_int64(128),
                              C.c_int64(128), p(ok), p(ok), p(ok), p(ok + 1), p(ok), 0, null, C.c_int64(0), null,
                              null) == sp.INVALID_ARG
    # spectra_decode: odd cache address
    assert lib.spectra_decode(C.byref(cfg), 0, p(ok + 1), p(ok), C.c_int64(1), C.c_int64(1), p(ok), 128, p(ok), p(ok),
                              p(ok), p(ok), sp.F32, null, C.c_int64(128 * 128), C.c_int64(128), null, C.c_int64(0),
                              null, null) == sp.INVALID_ARG
    # spectra_decode_attention: W_dec,K four bytes off
    big = C.c_size_t(1 << 30)
    assert lib.spectra_decode_attention(C.byref(cfg), p(ok), sp.F32, 1, 1, 4, p(ok), 128, p(ok), p(ok), p(ok), p(ok),
                                        C.c_int64(1), p(ok + 4), null, p(ok), p(ok), p(ok), p(ok), null, null,
                                        C.c_float(0), p(ok), sp.F32, null, p(ok), big, null, null, C.c_int64(0), null,
                                        null) == sp.INVALID_ARG


def test_cache_bytes_and_attention_path(lib):
    """Host helpers: a unit-side's buffer size for a capacity in tokens, and which kernels an attention call will
    run for a set of widths (the tensor-core kernels take every width profile at scale group 64 when the host copy of
    the widths is given; other scale groups and calls without host widths take the CUDA-core kernel)."""
    import numpy as np
    cfg = sp.default_config()
    w4 = [4] * 128
    assert sp.cache_bytes(cfg, w4, 0) == 0
    assert sp.cache_bytes(cfg, w4, 1) == sp.tile_bytes(cfg, w4)
    assert sp.cache_bytes(cfg, w4, 128) == sp.tile_bytes(cfg, w4)
    assert sp.cache_bytes(cfg, w4, 129) == 2 * sp.tile_bytes(cfg, w4)
    assert sp.cache_bytes(cfg, w4, 32768 + 64) == 257 * 9216
    assert sp.cache_bytes(cfg, [9] * 128, 128) == 0                                   # bad widths
    two = np.full((1, 128), 2, np.uint8)                                             # 8 blocks of 2-bit strips
    assert sp.attention_path(cfg, 8, 32, 1, two, two) == sp.PATH_TENSOR_CORE
    assert sp.attention_path(cfg, 4, 28, 1, two, two) == sp.PATH_TENSOR_CORE        # groups of 7 heads: two passes
    assert sp.attention_path(cfg, 8, 32, 1, None, None) == sp.PATH_CUDA_CORE        # no host widths
    assert sp.attention_path(sp.default_config(scale_group=32), 8, 32, 1, two, two) == sp.PATH_CUDA_CORE
    eight = np.full((1, 128), 8, np.uint8)
    assert sp.attention_path(cfg, 8, 32, 1, two, eight) == sp.PATH_TENSOR_CORE
    assert sp.attention_path(cfg, 8, 32, 1, eight, two) == sp.PATH_TENSOR_CORE
    seven = np.full((1, 128), 7, np.uint8)                                           # three sub-fields per channel
    assert sp.attention_path(cfg, 8, 32, 1, seven, seven) == sp.PATH_TENSOR_CORE
    with pytest.raises(sp.SpectraError):
        sp.attention_path(cfg, 3, 8, 1, two, two)
    with pytest.raises(sp.SpectraError):
        sp.attention_path(cfg, 8, 32, 1, two, np.full((1, 128), 9, np.uint8))


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(sp, "_lib", None)
    monkeypatch.setattr(sp, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(sp.SpectraError):
        sp.lib()
