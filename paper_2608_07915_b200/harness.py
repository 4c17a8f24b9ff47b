"""Device-resident coded KV cache for a whole model shape, driven through the C ABI.

Plumbing only (buffers, offsets, call order); used by bench.py and by the full-size parity tests so that
both exercise the same launch configuration.  Nothing here computes codec arithmetic.
"""
import numpy as np
import torch

import paper_2608_07915_b200 as sp
import spectra_inputs as si


class LayerSide:
    __slots__ = ("w_enc", "w_dec", "m_rot", "var", "widths", "widths_host", "tile_bytes", "cache", "unit_offset",
                 "unit_offset_host")


class CodedModelCache:
    """Coded K/V caches for `layers` layers, units ordered [sequence][kv-head] inside a layer, one parameter set
    per (layer, kv-head, side) fitted on the first n_fit tokens of sequence 0."""

    def __init__(self, wl, cfg=None, layers=None, batch=None, n_tokens=None, extra_tokens=256, device="cuda",
                 keep_raw_units=None):
        self.wl = wl
        self.cfg = cfg or sp.default_config()
        self.layers = wl.layers if layers is None else layers
        self.batch = wl.batch if batch is None else batch
        self.n_tokens = wl.n_tokens if n_tokens is None else n_tokens
        self.cap_tokens = self.n_tokens + extra_tokens
        self.cap_tiles = (self.cap_tokens + 127) // 128
        self.device = device
        self.H, self.Hq, self.d = wl.kv_heads, wl.q_heads, wl.head_dim
        self.n_units = self.batch * self.H
        self.side = [[None, None] for _ in range(self.layers)]
        self.seq_len = torch.zeros(self.batch, dtype=torch.int32, device=device)
        self.pos0 = torch.zeros(self.n_units, dtype=torch.int32, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.tensor_path = True                          # pass host widths to spectra_decode_attention
        self.keep_raw_units = keep_raw_units or {}      # {(layer, side): [unit indices]} raw vectors kept on host
        self.raw = {}
        self.timings = {}
        self.workspace = torch.zeros(
            max(16, sp.attention_workspace_bytes(self.cfg, self.batch, self.H, self.Hq, self.cap_tokens)),
            dtype=torch.uint8, device=device)

    # ------------------------------------------------------------------ set-up (calibrate + prefill encode)
    def draw_layer_side(self, layer, side):
        wl = self.wl
        dt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
        x = torch.empty((self.batch, self.H, self.n_tokens, self.d), dtype=dt, device=self.device)
        for h in range(self.H):
            x[:, h] = si.draw_unit_torch(wl, layer, h, side, self.batch, self.n_tokens, self.device)
        return x

    def build(self, time_phases=False, params_override=None):
        """params_override: optional {(layer, side): dict(w_enc, w_dec, m_rot, widths)} of numpy arrays [H, ...]; the
        library's own fit and allocation are skipped for those layer-sides (used by parity tests, which hand the
        same parameters to both implementations)."""
        cfg, H, d, N = self.cfg, self.H, self.d, self.n_tokens
        n_fit = min(self.wl.n_fit, N)
        f32 = dict(dtype=torch.float32, device=self.device)
        ev = lambda: torch.cuda.Event(enable_timing=True)
        t_fit = t_enc = 0.0
        sides = [(layer, side) for layer in range(self.layers) for side in (si.SIDE_K, si.SIDE_V)]
        n_ls = len(sides)
        w_enc_all, w_dec_all = (torch.zeros((n_ls * H, d, d), **f32) for _ in range(2))
        m_rot_all, var_all = (torch.zeros((n_ls * H, d), **f32) for _ in range(2))
        widths_all = torch.zeros((n_ls * H, d), dtype=torch.uint8, device=self.device)
        if any((params_override or {}).get(ls_key) is None for ls_key in sides):
            # calibration of the whole model in one call: the fit tokens (sequence 0 of every layer, head and side)
            # are gathered first, so that the per-matrix eigensolver CTAs fill the GPU
            dt = torch.bfloat16 if self.wl.dtype == "bf16" else torch.float32
            fit_x = torch.empty((n_ls * H, n_fit, d), dtype=dt, device=self.device)
            for i, (layer, side) in enumerate(sides):
                x = self.draw_layer_side(layer, side)
                fit_x[i * H:(i + 1) * H] = x[0, :, :n_fit]
                del x
            fit_ws = torch.zeros(sp.fit_workspace_bytes(cfg, n_ls * H), dtype=torch.uint8, device=self.device)
            e0, e1 = ev(), ev()
            e0.record()
            sp.fit_basis(cfg, fit_x, n_ls * H, n_fit, n_fit * d, d, w_enc_all, w_dec_all, m_rot_all, var_all, None, None,
                         fit_ws)
            sp.alloc_bits(cfg, var_all, n_ls * H, self.wl.ratio, widths_all)
            e1.record()
            torch.cuda.synchronize()
            t_fit = e0.elapsed_time(e1)
            del fit_x, fit_ws
        for i, (layer, side) in enumerate(sides):
            x = self.draw_layer_side(layer, side)
            ls = LayerSide()
            ls.w_enc, ls.w_dec = w_enc_all[i * H:(i + 1) * H], w_dec_all[i * H:(i + 1) * H]
            ls.m_rot, ls.var = m_rot_all[i * H:(i + 1) * H], var_all[i * H:(i + 1) * H]
            ls.widths = widths_all[i * H:(i + 1) * H]
            e1, e2 = ev(), ev()
            ov = (params_override or {}).get((layer, side))
            if ov is not None:
                ls.w_enc.copy_(torch.from_numpy(np.ascontiguousarray(ov["w_enc"], np.float32)))
                ls.w_dec.copy_(torch.from_numpy(np.ascontiguousarray(ov["w_dec"], np.float32)))
                ls.m_rot.copy_(torch.from_numpy(np.ascontiguousarray(ov["m_rot"], np.float32)))
                ls.widths.copy_(torch.from_numpy(np.ascontiguousarray(ov["widths"], np.uint8)))
            ls.widths_host = ls.widths.cpu().numpy()
            ls.tile_bytes = np.array([sp.tile_bytes(cfg, w) for w in ls.widths_host], np.int64)
            sizes = np.array([ls.tile_bytes[u % H] * self.cap_tiles for u in range(self.n_units)], np.int64)
            ls.unit_offset_host = np.concatenate([[0], np.cumsum(sizes)[:-1]]).astype(np.int64)
            ls.unit_offset = torch.from_numpy(ls.unit_offset_host).to(self.device)
            ls.cache = torch.empty(int(sizes.sum()), dtype=torch.uint8, device=self.device)
            self.pos0.zero_()
            e1.record()
            sp.encode(cfg, side, x, 0, self.n_units, H, self.pos0, N, N * d, d, ls.w_enc, ls.m_rot, ls.widths,
                      ls.cache, ls.unit_offset, self.status)
            e2.record()
            torch.cuda.synchronize()
            t_enc += e1.elapsed_time(e2)
            for u in self.keep_raw_units.get((layer, side), []):
                self.raw[(layer, side, u)] = x[u // H, u % H].float().cpu().numpy()
            self.side[layer][side] = ls
            del x
        self.seq_len.fill_(N)
        self.pos0.fill_(N)
        self.timings = dict(fit_alloc_ms=t_fit, prefill_encode_ms=t_enc)
        st = int(self.status.item())
        if st:
            raise sp.SpectraError(f"status word after prefill encode: {st}")
        return self

    # ------------------------------------------------------------------ one decode step of the whole model
    def append(self, layer, new_k, new_v):
        """new_k/new_v: [n_units, d] device tensors; appended at pos0 (not advanced here)."""
        cfg, H, d = self.cfg, self.H, self.d
        for side, x in ((si.SIDE_K, new_k), (si.SIDE_V, new_v)):
            ls = self.side[layer][side]
            sp.encode(cfg, side, x, 0, self.n_units, H, self.pos0, 1, d, d, ls.w_enc, ls.m_rot, ls.widths, ls.cache,
                      ls.unit_offset, self.status)

    def attend(self, layer, q, out, lse=None):
        k, v = self.side[layer]
        sp.decode_attention(self.cfg, q, self.batch, self.H, self.Hq, self.seq_len, self.cap_tokens, k.cache,
                            k.unit_offset, v.cache, v.unit_offset, self.H, k.w_dec, k.m_rot, k.widths, v.w_dec,
                            v.m_rot, v.widths, 0.0, out, lse, self.workspace, self.status,
                            k.widths_host if self.tensor_path else None, v.widths_host if self.tensor_path else None)

    def step_layer(self, layer, q, new_k, new_v, out, lse=None):
        """The fused call: append one token per unit at seq_len - 1 (seq_len already advanced) and attend."""
        k, v = self.side[layer]
        sp.decode_step(self.cfg, q, new_k, new_v, self.batch, self.H, self.Hq, self.seq_len, self.cap_tokens, k.cache,
                       k.unit_offset, v.cache, v.unit_offset, self.H, k.w_enc, k.w_dec, k.m_rot, k.widths, v.w_enc,
                       v.w_dec, v.m_rot, v.widths, 0.0, out, lse, self.workspace, self.status,
                       k.widths_host if self.tensor_path else None, v.widths_host if self.tensor_path else None)

    def decode_step(self, q_all, new_k_all, new_v_all, out_all, on_attend=None, fused=True):
        """q_all [layers, batch, Hq, d]; new_*_all [layers, n_units, d]; out_all like q_all.  Appends one token
        per sequence in every layer, then attends over the grown cache; advances the lengths at the end.  With
        fused=True a layer is one spectra_decode_step call, else spectra_encode (K, V) + spectra_decode_attention."""
        self.seq_len += 1
        for layer in range(self.layers):
            if on_attend:
                on_attend(layer, 0)
            if fused:
                self.step_layer(layer, q_all[layer], new_k_all[layer], new_v_all[layer], out_all[layer])
            else:
                self.append(layer, new_k_all[layer], new_v_all[layer])
                self.attend(layer, q_all[layer], out_all[layer])
            if on_attend:
                on_attend(layer, 1)
        self.pos0 += 1

    # ------------------------------------------------------------------ accounting
    def attention_bytes(self, layer=None):
        """Algorithmic bytes one decode-attention call reads and writes: every addressed K and V tile (payload +
        metadata) plus q and out."""
        n_tiles = (int(self.seq_len.max().item()) + 127) // 128
        layers = range(self.layers) if layer is None else [layer]
        total = 0
        for l in layers:
            for s in (0, 1):
                ls = self.side[l][s]
                total += int(sum(ls.tile_bytes[u % self.H] for u in range(self.n_units))) * n_tiles
            total += 2 * self.batch * self.Hq * self.d * 2
        return total

    def coded_bytes(self):
        return sum(self.side[l][s].cache.numel() for l in range(self.layers) for s in (0, 1))
