"""CPU oracle (test infrastructure): many-query causal attention over a reconstructed cache.

Mode A of Sec. 3.3 (reconstruct, then attend) for a chunk of new queries: every token of the unit is rebuilt by the
decoder (`oracle.codec.decode_unit`), optionally rounded to the storage type the attention reads (bfloat16), and query
i of the chunk, which sits at position pos0 + i, attends tokens 0 .. pos0 + i with the softmax written out in fp64.
Nothing here is blocked, fused or reordered; the decoder is the C oracle's.
"""
import numpy as np

from . import codec


def round_bf16(x):
    """fp64/fp32 -> the nearest bfloat16 (ties to even), returned as fp64.  Finite inputs only."""
    a = np.ascontiguousarray(x, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape).astype(np.float64)


def causal_attention(q, k, v, pos0, scale):
    """q [n_new, G, d]; k, v [n, d] with n >= pos0 + n_new.  Query i attends tokens 0 .. pos0 + i.

    Returns out [n_new, G, d] and lse [n_new, G] (natural logarithm of the sum of exp(scale q.k)), fp64.
    """
    q = np.asarray(q, np.float64)
    k = np.asarray(k, np.float64)
    v = np.asarray(v, np.float64)
    n_new, G, d = q.shape
    out = np.zeros((n_new, G, d))
    lse = np.zeros((n_new, G))
    for i in range(n_new):
        m = pos0 + i + 1
        for h in range(G):
            s = scale * (k[:m] @ q[i, h])
            top = s.max()
            e = np.exp(s - top)
            z = e.sum()
            out[i, h] = (e / z) @ v[:m]
            lse[i, h] = top + np.log(z)
    return out, lse


def reconstruct_unit(cache, tile_stride, n, w_dec, m_rot, widths, gs, side, storage="f64", rope=None):
    """The unit's n reconstructed vectors [n, d]; storage 'bf16' rounds them as the attention's input buffer does.
    rope = (theta,) applies the position rotation to the rebuilt vectors (keys), token t at position t."""
    if rope is None:
        _, xhat = codec.decode_unit(cache, tile_stride, n, w_dec, m_rot, widths, gs, side)
    else:
        xhat = codec.decode_unit_rope(cache, tile_stride, n, w_dec, m_rot, widths, gs, side, 0, rope[0])
    xhat = np.asarray(xhat, np.float64)
    return round_bf16(xhat) if storage == "bf16" else xhat


def prefill_mode_a(q, pos0, cache_k, stride_k, cache_v, stride_v, w_dec_k, m_rot_k, widths_k, w_dec_v, m_rot_v, widths_v,
                   gs, scale, storage="f64", rope=None):
    """One unit (sequence, KV head): q [n_new, G, d] are the queries of the G heads of its group for the chunk's
    n_new positions pos0 .. pos0 + n_new - 1; the coded caches hold pos0 + n_new tokens."""
    n = pos0 + np.asarray(q).shape[0]
    k = reconstruct_unit(cache_k, stride_k, n, w_dec_k, m_rot_k, widths_k, gs, codec.SIDE_K, storage, rope)
    v = reconstruct_unit(cache_v, stride_v, n, w_dec_v, m_rot_v, widths_v, gs, codec.SIDE_V, storage)
    return causal_attention(q, k, v, pos0, scale)
