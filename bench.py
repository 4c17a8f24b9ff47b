#!/usr/bin/env python
"""Benchmark of the SPECTRA coded-KV decode path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama32] [--impl ours|reference]

A step is one decode step of the whole model shape: in every layer, append one new token per sequence to the
coded K and V caches (rotate, quantise, pack) and run coded-cache decode attention over the grown cache.
Calibration (basis fit, bit allocation) and the prefill encode happen once during set-up and are reported
separately.  Prints one JSON line.  With --impl reference the CPU oracle is timed instead (a deliberately plain
program: a reported baseline, not a target).
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "coded_kv_decode_attention_kv_tokens_per_s"
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel (one layer of the workload),
# from the ncu capture summarised in profiles/attention_mma_kernel_llama32_2layer.md (same per-launch shape)
NCU_TRAFFIC_BYTES = {"llama32": 172.8e6}
# share of the dominant kernel (attention_mma_kernel) in the device time of a decode step, from the launch list of
# this command summarised in profiles/decode_step_launch_list_llama32.md
MAIN_KERNEL_SHARE = {"llama32": 0.778}
UNIT = "KV tokens/s"
MIN_TIMED_SECONDS = 0.5      # the --steps set is repeated until the timed region is at least this long
# what the metric's path computes in: codes and probabilities enter mma.sync as fp16 (codes exactly, the query as
# a hi + lo pair), sums are fp32
ARITHMETIC = "f16xf16->f32"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def _tensor_peak():
    """Dense bf16 TFLOP/s of a library GEMM timed alone on this machine (the burst figure), else the fallback."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["bf16_tflops"]), "measured"
    return 1590.0, "fallback"


class ClockSampler:
    """Samples SM clocks and clock-event reasons of one GPU in a background thread (NVML, read-only)."""

    REASONS = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40}

    def __init__(self, gpu_index, period_s=0.01):
        import threading
        self.idx, self.period = gpu_index, period_s
        self.sm, self.reasons, self.max_sm = [], set(), None
        self._stop = threading.Event()
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._ok = False

    def _run(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            # honour CUDA_VISIBLE_DEVICES when it lists indices
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            phys = self.idx
            if vis and all(v.strip().isdigit() for v in vis.split(",")):
                phys = int(vis.split(",")[self.idx])
            h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_sm = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            self._ok = True
            while not self._stop.is_set():
                self.sm.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                try:
                    mask = int(pynvml.nvmlDeviceGetCurrentClocksEventReasons(h))
                except Exception:
                    mask = int(pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                for name, bit in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
                time.sleep(self.period)
        except Exception:
            self._ok = False

    def start(self):
        self._thread.start()

    def stop(self):
        self._stop.set()
        self._thread.join(timeout=5)
        out = {"sm_mhz": None, "sm_max_mhz": self.max_sm, "reasons": sorted(self.reasons), "samples": len(self.sm)}
        if self.sm:
            out["sm_mhz"] = float(np.median(self.sm))
        return out


def _dist_setup(n_gpus):
    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    return rank, world, local


def _barrier(world):
    import torch
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()


def _max_over_ranks(x, world, device="cuda"):
    import torch
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# ---------------------------------------------------------------------------------------------- CPU oracle legs

class OracleSample:
    """A bounded sample of the workload built and run by the oracle alone (numpy generator, oracle fit,
    allocation and encode): `heads` kv-heads of layer 0, sequence 0, n_tokens cached tokens."""

    def __init__(self, wl, n_tokens):
        import spectra_inputs as si
        from oracle import codec as oc
        from oracle import fit as ofit
        self.wl, self.n, self.oc = wl, n_tokens, oc
        H, d = wl.kv_heads, wl.head_dim
        self.G = wl.q_heads // H
        self.par = {}
        cap_tiles = (n_tokens + 1 + 127) // 128
        for side in (si.SIDE_K, si.SIDE_V):
            X = np.stack([si.draw_unit(wl, 0, h, side, 0, n_tokens=n_tokens) for h in range(H)])
            fits = [ofit.fit_basis(X[h][:min(wl.n_fit, n_tokens)].astype(np.float64), ofit.GAIN_SQRT) for h in range(H)]
            widths = np.stack([ofit.alloc_bits(f["v_alloc"].astype(np.float32), ofit.total_bits(d, wl.ratio))
                               for f in fits])
            tb = np.array([oc.tile_bytes(w, 64) for w in widths], np.int64)
            off = np.concatenate([[0], np.cumsum(tb * cap_tiles)[:-1]]).astype(np.int64)
            cache = np.zeros(int((tb * cap_tiles).sum()), np.uint8)
            we = np.stack([f["W_enc"] for f in fits]).astype(np.float32)
            wd = np.stack([f["W_dec"] for f in fits]).astype(np.float32)
            mr = np.stack([f["m_rot"] for f in fits]).astype(np.float32)
            oc.encode_units(X, we, mr, widths, 64, side, 0, cache, off, tb)
            self.par[side] = dict(we=we, wd=wd, mr=mr, widths=widths, tb=tb, off=off, cache=cache)
        self.q = si.draw_queries(wl, 0, 0).reshape(H, self.G, d).astype(np.float64)
        self.new = {side: np.stack([si.draw_unit(wl, 0, h, side, 0, n_tokens=1, start=n_tokens) for h in range(H)])
                    for side in (si.SIDE_K, si.SIDE_V)}

    def step(self):
        """One decode step on the sample: append one token per unit (both sides), then latent-space attention
        over n+1 tokens.  Returns (seconds, token_heads, threads)."""
        oc = self.oc
        k, v = self.par[0], self.par[1]
        H = self.wl.kv_heads
        t0 = time.perf_counter()
        for side in (0, 1):
            p = self.par[side]
            oc.encode_units(self.new[side], p["we"], p["mr"], p["widths"], 64, side, self.n, p["cache"], p["off"],
                            p["tb"])
        oc.attention_units("B", self.q, [self.n + 1] * H, k["cache"], k["off"], k["tb"], v["cache"], v["off"],
                           v["tb"], k["wd"], k["mr"], k["widths"], v["wd"], v["mr"], v["widths"], 64,
                           1.0 / np.sqrt(128.0))
        dt = time.perf_counter() - t0
        return dt, H * (self.n + 1), min(oc.num_threads(), H)


ORACLE_SAMPLE_TOKENS = 32768      # cached tokens per head of the oracle's sample, the same in both legs


def _oracle_rate(wl, reps=1, warm=0):
    """The oracle's fixed sample: all kv-heads of layer 0, sequence 0, min(context, 32768) cached tokens.  Runs
    warm + reps decode steps on it; returns (times of the reps, token_heads per step, threads, description)."""
    n = min(wl.n_tokens, ORACLE_SAMPLE_TOKENS)
    sample = OracleSample(wl, n)
    times = []
    th = threads = 0
    for i in range(warm + reps):
        dt, th, threads = sample.step()
        if i >= warm:
            times.append(dt)
    desc = (f"layer 0, sequence 0, {wl.kv_heads} kv-heads x {n} cached tokens, built and run by the oracle alone; "
            f"one step = append 1 token per unit + Mode B attention; token-heads/s divided by layers*kv_heads")
    return times, th, threads, desc


def run_reference(args, wl):
    """The reference arm: the CPU oracle, as it stands, on a bounded sample of the same workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times, th, threads, desc = _oracle_rate(wl, args.steps, args.warmup)
    t = float(np.mean(times))
    value = th / t / (wl.layers * wl.kv_heads)          # same unit as the GPU arm: KV tokens/s of the full model
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "note": "CPU oracle on a bounded sample; value scaled to the full model "
                                                "shape"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------- GPU arm

def run_ours(args, wl):
    import torch

    import paper_2608_07915_b200 as sp
    from paper_2608_07915_b200 import harness
    rank, world, local = _dist_setup(args.gpus)
    dev = torch.device("cuda", local)
    steps, warmup = args.steps, max(args.warmup, 3)
    hbm_gbs, peak_kind = _peaks()
    model = harness.CodedModelCache(wl, layers=args.layers or None,
                                    extra_tokens=(2 * args.max_repeats + 3) * steps + warmup + 64)
    t0 = time.perf_counter()
    model.build(time_phases=True)
    setup_s = time.perf_counter() - t0
    L, B, H, Hq, d, U = model.layers, model.batch, model.H, model.Hq, model.d, model.n_units
    dt = torch.bfloat16
    gen = torch.Generator(device="cuda").manual_seed(1234 + rank)
    n_in = 4                                           # distinct input sets, cycled
    q_dev = torch.randn((n_in, L, B, Hq, d), generator=gen, device="cuda").to(dt)
    nk_dev = torch.randn((n_in, L, U, d), generator=gen, device="cuda").to(dt)
    nv_dev = torch.randn((n_in, L, U, d), generator=gen, device="cuda").to(dt)
    out_dev = torch.zeros((L, B, Hq, d), dtype=dt, device="cuda")
    q_host, nk_host, nv_host = (t.cpu().pin_memory() for t in (q_dev, nk_dev, nv_dev))
    out_host = torch.zeros((L, B, Hq, d), dtype=dt).pin_memory()
    q_stage, nk_stage, nv_stage = (torch.empty_like(t[0]) for t in (q_dev, nk_dev, nv_dev))

    ev = lambda: torch.cuda.Event(enable_timing=True)
    attn_events = []

    def mark(layer, which):
        e = ev(); e.record(); attn_events.append(e)

    def step_resident(i, timed=False):
        model.decode_step(q_dev[i % n_in], nk_dev[i % n_in], nv_dev[i % n_in], out_dev, mark if timed else None,
                          fused=args.fused)

    e2e_graph = []                                     # the step on the staging buffers, captured once (graph mode)

    def step_e2e(i):
        q_stage.copy_(q_host[i % n_in], non_blocking=True)
        nk_stage.copy_(nk_host[i % n_in], non_blocking=True)
        nv_stage.copy_(nv_host[i % n_in], non_blocking=True)
        if e2e_graph:
            e2e_graph[0].replay()
        else:
            model.decode_step(q_stage, nk_stage, nv_stage, out_dev, fused=args.fused)
        out_host.copy_(out_dev, non_blocking=True)

    # ---- device-resident timing
    for i in range(warmup):
        step_resident(i)
    graphs = None
    if args.graph:
        # one CUDA graph per input set: the whole 32-layer step (appends, prep, main, combine, length updates)
        torch.cuda.synchronize()
        graphs = []
        for k in range(n_in):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                step_resident(k)
            graphs.append(g)
        for k in range(n_in):
            graphs[k].replay()
    # the --steps set is repeated so that the timed region lasts at least MIN_TIMED_SECONDS (one untimed set sizes it)
    _barrier(world)
    p0, p1 = ev(), ev()
    p0.record()
    for i in range(steps):
        if graphs:
            graphs[i % n_in].replay()
        else:
            step_resident(i)
    p1.record()
    torch.cuda.synchronize()
    repeats = int(max(1, min(args.max_repeats, np.ceil(MIN_TIMED_SECONDS * 1e3 / max(p0.elapsed_time(p1), 1e-3)))))
    repeats = int(_max_over_ranks(float(repeats), world))
    _barrier(world)
    sampler = ClockSampler(local)
    sampler.start()
    marks = [ev() for _ in range(repeats + 1)]
    marks[0].record()
    for r in range(repeats):
        for i in range(steps):
            if graphs:
                graphs[i % n_in].replay()
            else:
                step_resident(i, timed=True)
        marks[r + 1].record()
    _barrier(world)
    ms_step = _max_over_ranks(marks[0].elapsed_time(marks[repeats]) / (steps * repeats), world)
    ms_step_sets = [marks[r].elapsed_time(marks[r + 1]) / steps for r in range(repeats)]
    if graphs:
        # events cannot be recorded inside a replayed graph: time the attention calls of the same steps, launched
        # directly, right after the timed region (same buffers, same lengths + 1 per step)
        for i in range(min(steps, 4)):
            step_resident(i, timed=True)
        torch.cuda.synchronize()
    clocks = sampler.stop()
    attn_ms = [attn_events[2 * j].elapsed_time(attn_events[2 * j + 1]) for j in range(len(attn_events) // 2)]
    attn_ms_avg = float(np.mean(attn_ms))
    n_ctx = int(model.seq_len.max().item())
    kv_tokens = B * n_ctx

    # ---- end to end: pinned host inputs copied in, outputs copied out, every step
    for i in range(2):
        step_e2e(i)
    if args.graph:
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            model.decode_step(q_stage, nk_stage, nv_stage, out_dev, fused=args.fused)
        e2e_graph.append(g)
        step_e2e(2)
    _barrier(world)
    e0, e1 = ev(), ev()
    e0.record()
    for i in range(steps * repeats):
        step_e2e(i)
    e1.record()
    _barrier(world)
    ms_e2e = _max_over_ranks(e0.elapsed_time(e1) / (steps * repeats), world)
    status = int(model.status.item())

    # ---- reconstruction (spectra_decode) of one layer's K side, outside the timed decode steps: reported beside
    # the prefill encode as a phase figure
    ls0 = model.side[0][0]
    n_tok = torch.full((U,), wl.n_tokens, dtype=torch.int32, device="cuda")
    recon = torch.empty((U, wl.n_tokens, d), dtype=torch.bfloat16, device="cuda")
    # one warm-up call, then four calls launched back to back between two events (the device is never left waiting for
    # the host to prepare the next launch): time per call
    n_rec_calls = 4
    for k in range(1 + n_rec_calls):
        if k == 1:
            torch.cuda.synchronize()
            r0, r1 = ev(), ev()
            r0.record()
        sp.decode(model.cfg, 0, ls0.cache, ls0.unit_offset, U, H, n_tok, wl.n_tokens, ls0.w_dec, ls0.m_rot,
                  ls0.widths, recon, None, wl.n_tokens * d, d)
    r1.record()
    torch.cuda.synchronize()
    del recon
    reconstruct_ms = r0.elapsed_time(r1) / n_rec_calls

    # bulk encode: raw vectors read (2 B each) + packed tiles written; reconstruction: packed tiles read + bf16 written
    tile_bytes_all = sum(int(model.side[l][sd].tile_bytes[u % H]) for l in range(L) for sd in (0, 1) for u in range(U))
    enc_bytes = L * 2 * U * wl.n_tokens * d * 2 + tile_bytes_all * (wl.n_tokens // 128)
    rec_bytes = U * wl.n_tokens * d * 2 + sum(int(ls0.tile_bytes[u % H]) for u in range(U)) * (wl.n_tokens // 128)
    bytes_call = model.attention_bytes(layer=0)
    # duration of one launch of the dominant kernel inside the timed region: the step's device time per layer times
    # the kernel's share of a step in the committed launch list; the directly launched layer call (front + main +
    # combine between two events) is kept beside it
    share = MAIN_KERNEL_SHARE.get(wl.name)
    ms_launch = ms_step / L * share if share else attn_ms_avg
    achieved = bytes_call / (ms_launch * 1e-3) / 1e9
    h2d = sum(t[0].numel() * t.element_size() for t in (q_host, nk_host, nv_host))
    d2h = out_host.numel() * out_host.element_size()
    line = {
        "metric": METRIC, "value": world * kv_tokens / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": steps, "repeats": repeats, "warmup": warmup, "ms_per_step": ms_step,
        "ms_per_step_median_of_sets": float(np.median(ms_step_sets)), "timed_region_s": ms_step * steps * repeats * 1e-3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": ARITHMETIC, "data": "synthetic",
        "config": {"workload": wl.name, "layers": L, "batch": B, "kv_heads": H, "q_heads": Hq, "head_dim": d,
                   "context": n_ctx, "ratio": wl.ratio, "cache_dtype_replaced": "bf16",
                   "coded_cache_gb": model.coded_bytes() / 1e9, "parallelism": f"replicas{world}",
                   "launch": "cuda_graph_per_step" if graphs else "direct",
                   "l2": "coded cache per step far exceeds L2; no flush needed" if model.coded_bytes() > 4e8
                   else "WARNING: coded cache fits L2"},
        "e2e": {"value": world * kv_tokens / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e},
        "gpu_launches": steps * repeats * L * (sp.STEP_LAUNCHES if args.fused else 2 + sp.ATTENTION_LAUNCHES),
        "clocks": clocks,
        "roofline": {"bound": "hbm", "kernel": "attention_mma_kernel (one launch = one layer of the step)",
                     "achieved": achieved, "peak": hbm_gbs, "unit": "GB/s", "frac": achieved / hbm_gbs,
                     "peak_kind": peak_kind, "traffic": NCU_TRAFFIC_BYTES.get(wl.name), "bytes_per_launch": bytes_call,
                     "ms_per_launch": ms_launch,
                     "ms_per_launch_from": "ms_per_step / layers * main_kernel_share" if share else "direct layer call",
                     "main_kernel_share": share,
                     "layer_call_direct_ms": attn_ms_avg,
                     "layer_call_direct_frac": bytes_call / (attn_ms_avg * 1e-3) / 1e9 / hbm_gbs,
                     "whole_step_frac": bytes_call * L / (ms_step * 1e-3) / 1e9 / hbm_gbs},
        "phases": {"setup_s": setup_s, "fit_alloc_ms_total": model.timings["fit_alloc_ms"],
                   "prefill_encode_ms_total": model.timings["prefill_encode_ms"],
                   "prefill_encode_tokens_per_s": L * 2 * U * wl.n_tokens / max(model.timings["prefill_encode_ms"],
                                                                               1e-9) * 1e3 / 2,
                   "reconstruct_ms_per_layer_side": reconstruct_ms,
                   "reconstruct_unit_tokens_per_s": U * wl.n_tokens / max(reconstruct_ms, 1e-9) * 1e3,
                   # algorithmic bytes of the two bulk phases against the same HBM peak (both are far from it: their
                   # scalar quantise / pack / unpack phases bound them)
                   "prefill_encode_gbs": enc_bytes / max(model.timings["prefill_encode_ms"], 1e-9) / 1e6,
                   "prefill_encode_frac_of_hbm": enc_bytes / max(model.timings["prefill_encode_ms"], 1e-9) / 1e6 / hbm_gbs,
                   "reconstruct_gbs": rec_bytes / max(reconstruct_ms, 1e-9) / 1e6,
                   "reconstruct_frac_of_hbm": rec_bytes / max(reconstruct_ms, 1e-9) / 1e6 / hbm_gbs},
        "status_word": status,
    }
    if rank == 0 and world == 1 and args.other_workloads and not args.layers:
        del model, q_dev, nk_dev, nv_dev
        torch.cuda.empty_cache()
        line["other_workloads"] = _other_workloads(args, hbm_gbs)
        line["prefill_attention"] = _prefill_attention()
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        times, th, threads, desc = _oracle_rate(wl, 3, 1)
        line["cpu_baseline"] = {"value": th / float(np.mean(times)) / (wl.layers * wl.kv_heads), "unit": UNIT,
                                "cores": threads, "kind": "oracle", "sample": desc}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def _other_workloads(args, hbm_gbs):
    """One layer of each other workload shape: the fused layer call (front + main + combine) launched directly and
    timed with CUDA events, the L2 flushed before every timed call (one layer's coded cache can fit the L2)."""
    import torch

    import spectra_inputs as si
    from paper_2608_07915_b200 import harness
    out = {}
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    ev = lambda: torch.cuda.Event(enable_timing=True)
    for name in ("llama1", "qwen28", "long128k", "batch32"):
        wl = si.WORKLOADS[name]
        n_calls, n_warm = 10, 3
        m = harness.CodedModelCache(wl, layers=1, extra_tokens=n_calls + n_warm + 8)
        m.build()
        L, B, Hq, d, U = 1, m.batch, m.Hq, m.d, m.n_units
        gen = torch.Generator(device="cuda").manual_seed(4321)
        q = torch.randn((1, B, Hq, d), generator=gen, device="cuda").to(torch.bfloat16)
        nk = torch.randn((1, U, d), generator=gen, device="cuda").to(torch.bfloat16)
        nv = torch.randn((1, U, d), generator=gen, device="cuda").to(torch.bfloat16)
        o = torch.zeros((1, B, Hq, d), dtype=torch.bfloat16, device="cuda")
        ms = []
        for i in range(n_warm + n_calls):
            flush.zero_()
            e0, e1 = ev(), ev()
            e0.record()
            m.decode_step(q, nk, nv, o, fused=True)
            e1.record()
            torch.cuda.synchronize()
            if i >= n_warm:
                ms.append(e0.elapsed_time(e1))
        b = m.attention_bytes(layer=0)
        t = float(np.median(ms))
        out[name] = {"layers_timed": 1, "batch": B, "context": int(m.seq_len.max().item()), "ratio": wl.ratio,
                     "ms_per_layer_call": t, "bytes_per_layer_call": b, "frac_of_hbm": b / (t * 1e-3) / 1e9 / hbm_gbs,
                     "status_word": int(m.status.item()), "l2": "flushed before every timed call"}
        del m, q, nk, nv, o
        torch.cuda.empty_cache()
    return out


def _prefill_attention(n_new=32768, reps=5):
    """The many-query path (reconstruct, then attend): causal attention of one 32768-token chunk over reconstructed
    bf16 page pools in the Llama-3.1-8B head shape, one layer, timed alone with CUDA events.  The pools hold seeded
    random values (the kernel's speed does not depend on them); flops are the algorithmic ones of causal attention,
    4 d per (query, visible token) pair, against the measured dense bf16 peak of a library GEMM."""
    import torch

    import paper_2608_07915_b200 as sp
    n_seq, Hq, Hkv, d = 1, 32, 8, 128
    tiles = (n_new + 127) // 128
    n_pages = n_seq * Hkv * tiles
    gen = torch.Generator(device="cuda").manual_seed(99)
    kp = torch.randn((n_pages, 128, d), generator=gen, device="cuda").to(torch.bfloat16)
    vp = torch.randn((n_pages, 128, d), generator=gen, device="cuda").to(torch.bfloat16)
    q = torch.randn((n_seq, n_new, Hq, d), generator=gen, device="cuda").to(torch.bfloat16)
    out = torch.empty_like(q)
    pos0 = torch.zeros(n_seq, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    strides = (n_new * Hq * d, Hq * d, d)
    ms = []
    for i in range(3 + reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        sp.prefill_attention(q, kp, vp, n_pages, 128 * d, d, None, tiles, n_seq, Hkv, Hq, pos0, n_new, strides,
                             1.0 / np.sqrt(d), out, strides, None, status)
        e1.record()
        torch.cuda.synchronize()
        if i >= 3:
            ms.append(e0.elapsed_time(e1))
    t = float(np.median(ms))
    flops = 4.0 * d * n_seq * Hq * (n_new * (n_new + 1) // 2)
    peak, kind = _tensor_peak()
    return {"workload": f"{n_seq} sequence x {n_new} new tokens, {Hq} query / {Hkv} KV heads, head_dim {d}, bf16 pools",
            "kernel": "prefill_attention_kernel", "ms": t, "bound": "tensor", "achieved": flops / (t * 1e-3) / 1e12,
            "peak": peak, "unit": "TFLOP/s", "frac": flops / (t * 1e-3) / 1e12 / peak, "peak_kind": kind,
            "flops": flops, "status_word": int(status.item())}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="llama32")
    ap.add_argument("--layers", type=int, default=0, help="debug: fewer layers than the workload (invalid as a result)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-workloads", dest="other_workloads", action="store_false",
                    help="skip the one-layer timings of the other workload shapes")
    ap.add_argument("--max-repeats", type=int, default=64, help="upper bound of the repeats of the --steps set")
    ap.add_argument("--unfused", dest="fused", action="store_false",
                    help="per layer: spectra_encode (K, V) + spectra_decode_attention instead of spectra_decode_step")
    ap.add_argument("--prefill-only", action="store_true",
                    help="time only the many-query attention over reconstructed pools and print its record")
    ap.add_argument("--prefill-tokens", type=int, default=32768, help="chunk length of --prefill-only")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="launch the timed steps directly instead of replaying them as CUDA graphs")
    args = ap.parse_args()
    if args.prefill_only:
        print(json.dumps({"prefill_attention": _prefill_attention(args.prefill_tokens, reps=2)}), flush=True)
        return
    import spectra_inputs as si
    wl = si.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
