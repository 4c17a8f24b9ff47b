"""The workspace-free calibration entry point (spectra_fit_basis_static) against the ordinary one.

Some callers of this library cannot allocate device memory at the moment they calibrate (a plug-in inside a host
process that owns a fixed memory arena, or a component started after the allocator was frozen).  For them the
library carries its calibration scratch in a fixed array of its own.  This file checks, through the C ABI, that the
variant writes what spectra_fit_basis writes, twice in a row (the array still holds the first call's contents when
the second starts), and that it refuses more unit-sides than the array holds.  It is collected last on purpose.
"""
import ctypes as C

import numpy as np
import pytest

import spectra_inputs as si

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _fit(sp, cfg, xd, n_units, n, static):
    f32 = dict(dtype=torch.float32, device="cuda")
    w_enc, w_dec, U = (torch.zeros((n_units, 128, 128), **f32) for _ in range(3))
    m_rot, var, lam = (torch.zeros((n_units, 128), **f32) for _ in range(3))
    if static:
        sp.fit_basis_static(cfg, xd, n_units, n, n * 128, 128, w_enc, w_dec, m_rot, var, lam, U)
    else:
        ws = torch.zeros(sp.fit_workspace_bytes(cfg, n_units), dtype=torch.uint8, device="cuda")
        sp.fit_basis(cfg, xd, n_units, n, n * 128, 128, w_enc, w_dec, m_rot, var, lam, U, ws)
    torch.cuda.synchronize()
    return [t.cpu().numpy().astype(np.float64) for t in (w_enc, w_dec, m_rot, var, lam, U)]


def test_static_scratch_fit_matches_workspace_fit_twice():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2608_07915_b200 as sp
    cfg = sp.default_config()
    wl = si.WORKLOADS["tiny"]
    n = 768
    for call, n_units in enumerate((3, sp.FIT_STATIC_MAX_UNITS)):        # second call: more units, dirty scratch
        X = np.stack([si.draw_unit(wl, 0, h + 10 * call, si.SIDE_K if h % 2 else si.SIDE_V, 0, n_tokens=n)
                      for h in range(n_units)])
        xd = torch.from_numpy(X).cuda()
        ref = _fit(sp, cfg, xd, n_units, n, static=False)
        got = _fit(sp, cfg, xd, n_units, n, static=True)
        lam1 = ref[4][:, :1]
        # the accumulation order of the fp64 sums differs between launches (atomics), so eigenvalues agree to
        # rounding, not bit for bit; eigenvectors of well separated eigenvalues agree to the same level
        assert np.abs(got[4] - ref[4]).max() <= 1e-6 * lam1.max()
        assert np.abs(got[3] - ref[3]).max() <= 1e-5 * np.abs(ref[3]).max()
        assert np.abs(got[2] - ref[2]).max() <= 1e-4 * np.abs(ref[2]).max() + 1e-6
        for u in range(n_units):
            Ug, Ur = got[5][u], ref[5][u]
            assert np.abs(Ug.T @ Ug - np.eye(128)).max() <= 5e-6
            # same leading subspace: the 16 strongest directions coincide (tails can rotate inside near-ties)
            assert np.abs(np.abs(Ug[:, :16].T @ Ur[:, :16]) - np.eye(16)).max() <= 1e-3
            assert np.abs(got[0][u] @ got[1][u] - np.eye(128)).max() <= 2e-5


def test_static_scratch_fit_rejects_oversized_calls():
    import paper_2608_07915_b200 as sp
    cfg = sp.default_config()
    null = C.c_void_p(0)
    rc = sp.lib().spectra_fit_basis_static(C.byref(cfg), null, 0, C.c_int64(sp.FIT_STATIC_MAX_UNITS + 1),
                                           C.c_int64(16), C.c_int64(0), C.c_int64(0), null, null, null, null, null,
                                           null, null)
    assert rc == sp.CAPACITY
