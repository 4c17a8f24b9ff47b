"""Seeded synthetic KV caches and queries shared by the tests, the smoke check and the benchmark.

This module holds no codec arithmetic: it only draws inputs.  The recipe stands in for the
long-context key/value caches of Llama-3.1-8B- and Qwen2.5-7B-shaped models (the paper's
Observation 1: correlated channels, strongly skewed energy, a few outlier channels):

    Q      = orthogonal factor of the QR of a d x d standard-normal matrix (diag(R) > 0)
    lam_i  = i^(-alpha), i = 1..d
    x      = (z * sqrt(lam)) Q^T,  z ~ N(0, I)        (covariance Q diag(lam) Q^T)
    then n_out seeded channel indices are multiplied by s_out

Every (layer, kv-head, side) has its own covariance; the sequences of a batch share it and
differ in z.  Seeds are SeedSequence([BASE, config, layer, head, side, seq]).
"""
from dataclasses import dataclass

import numpy as np

BASE_SEED = 20260807
SIDE_K, SIDE_V = 0, 1


@dataclass(frozen=True)
class SideRecipe:
    alpha: float
    n_out: int
    s_out: float


@dataclass(frozen=True)
class Workload:
    name: str
    config_id: int
    layers: int
    kv_heads: int
    q_heads: int
    batch: int
    n_tokens: int
    n_fit: int
    ratio: float
    dtype: str           # "f32" or "bf16"
    k: SideRecipe
    v: SideRecipe
    head_dim: int = 128

    @property
    def group(self):
        return self.q_heads // self.kv_heads


_K0 = SideRecipe(1.5, 4, 15.0)
_V0 = SideRecipe(1.0, 0, 1.0)

WORKLOADS = {
    "tiny": Workload("tiny", 0, 1, 1, 4, 1, 1024, 1024, 4.0, "f32", _K0, _V0),
    "llama1": Workload("llama1", 1, 1, 8, 32, 1, 32768, 4096, 4.0, "bf16", _K0, _V0),
    "llama32": Workload("llama32", 2, 32, 8, 32, 8, 32768, 4096, 8.0, "bf16", _K0, _V0),
    "qwen28": Workload("qwen28", 3, 28, 4, 28, 16, 65536, 4096, 12.0, "bf16", SideRecipe(2.0, 8, 20.0), _V0),
    "long128k": Workload("long128k", 4, 32, 8, 32, 1, 131072, 4096, 8.0, "bf16", _K0, _V0),
    "batch32": Workload("batch32", 4, 32, 8, 32, 32, 32768, 4096, 8.0, "bf16", _K0, _V0),
}


def _rng(*key):
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([BASE_SEED, *[int(k) for k in key]])))


def mixing_matrix(config_id, layer, head, side, recipe, d=128):
    """A [d, d] fp64 with x = z A for z ~ N(0, I): A = diag(sqrt(lam)) Q^T, outlier columns scaled."""
    rng = _rng(config_id, layer, head, side, 0xC0)
    g = rng.standard_normal((d, d))
    q, r = np.linalg.qr(g)
    q = q * np.sign(np.diag(r))[None, :]
    lam = np.arange(1, d + 1, dtype=np.float64) ** (-recipe.alpha)
    a = np.sqrt(lam)[:, None] * q.T
    if recipe.n_out:
        idx = rng.choice(d, size=recipe.n_out, replace=False)
        a[:, idx] *= recipe.s_out
    return a


def to_bf16_f32(x):
    """Round fp32 values to bf16 (nearest even), returned as fp32 (numpy has no bf16)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def draw_unit(wl, layer, head, side, seq, n_tokens=None, start=0):
    """Cache vectors [n_tokens, d] of one (layer, head, side, seq) as fp32 (bf16-representable when the
    workload dtype is bf16).  `start` offsets the token stream so appended tokens continue it."""
    n_tokens = wl.n_tokens if n_tokens is None else n_tokens
    recipe = wl.k if side == SIDE_K else wl.v
    a = mixing_matrix(wl.config_id, layer, head, side, recipe, wl.head_dim)
    rng = _rng(wl.config_id, layer, head, side, seq, start)
    z = rng.standard_normal((n_tokens, wl.head_dim))
    x = (z @ a).astype(np.float32)
    return to_bf16_f32(x) if wl.dtype == "bf16" else x


def mean_offset(wl, layer, head, side, scale=1.0):
    """A constant vector [d] fp32 to add to every cache vector of one (layer, head, side): +-scale standard
    deviations of each channel (seeded signs).  The recipe above is zero-mean; with this offset the rotated means
    the codec removes and restores are as large as the spread of the data."""
    recipe = wl.k if side == SIDE_K else wl.v
    a = mixing_matrix(wl.config_id, layer, head, side, recipe, wl.head_dim)
    sigma = np.sqrt((a * a).sum(axis=0))
    sign = _rng(wl.config_id, layer, head, side, 0x4D).choice([-1.0, 1.0], size=wl.head_dim)
    c = (scale * sign * sigma).astype(np.float32)
    return to_bf16_f32(c) if wl.dtype == "bf16" else c


def draw_queries(wl, layer, seq, step=0):
    """Decode queries [q_heads, d] fp32 (bf16-representable for bf16 workloads)."""
    rng = _rng(wl.config_id, layer, 0xAB, seq, step)
    q = rng.standard_normal((wl.q_heads, wl.head_dim)).astype(np.float32)
    return to_bf16_f32(q) if wl.dtype == "bf16" else q


def draw_unit_torch(wl, layer, head, side, n_seq, n_tokens, device, seed_extra=0):
    """GPU-side bulk draw for the large workloads: [n_seq, n_tokens, d] in the workload dtype.
    Same covariance recipe; z comes from torch's Philox generator (different stream from draw_unit)."""
    import torch
    recipe = wl.k if side == SIDE_K else wl.v
    a = torch.from_numpy(mixing_matrix(wl.config_id, layer, head, side, recipe, wl.head_dim)).to(
        device=device, dtype=torch.float32)
    gen = torch.Generator(device=device)
    gen.manual_seed((BASE_SEED * 1000003 + wl.config_id * 7919 + layer * 613 + head * 31 + side * 7 + seed_extra)
                    % (2 ** 62))
    z = torch.randn((n_seq, n_tokens, wl.head_dim), generator=gen, device=device, dtype=torch.float32)
    x = z @ a
    return x.to(torch.bfloat16) if wl.dtype == "bf16" else x
