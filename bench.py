#!/usr/bin/env python
"""Benchmark of the LogQuant decode hot path on B200.

One "step" = one decode step of a Llama-3-8B-shaped stack: for each of the L layer caches,
append the new token's K/V (running the window-overflow step when the bf16 window is full) and run
decode attention over the whole mixed cache.  Metric: KV tokens/s = B * (n_quant + n_fp) * L / t_step
summed over all ranks (independent replicas, no collective on the data path).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints ONE JSON line.  `--impl reference` times the CPU oracle (oracle/, as it stands) on the host
cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2503_19950_b200 import synth  # noqa: E402

WORKLOADS = {
    # the configuration the metric is quoted on: Llama-3-8B layer shape, batch 8, context 8192, W=128, G=32, 32 stacked layers
    "llama3-8b-8k": dict(L=32, B=8, Hq=32, Hkv=8, W=128, G=32, ctx=8192, n_outliers=3, seed=2),
    # config 2 in the paper's own setting (Sec. 3.1): group 64, reserved length 128 tokens, i.e. W = 42 (not a
    # multiple of G: removed tokens wait at full precision until 64 of them form a key group)
    "llama3-8b-8k-w42": dict(L=32, B=8, Hq=32, Hkv=8, W=42, G=64, ctx=8192, n_outliers=3, seed=2),
    # config 2 as a ragged batch: prompts of 8192, 7168, ..., 1024 tokens, left-padded to 8192 positions
    "llama3-8b-8k-ragged": dict(L=32, B=8, Hq=32, Hkv=8, W=128, G=32, ctx=8192, n_outliers=3, seed=2,
                                pad=[0, 1024, 2048, 3072, 4096, 5120, 6144, 7168]),
    # config 2 with the paper's second precision (4-bit codes, 160 B per token)
    "llama3-8b-8k-int4": dict(L=32, B=8, Hq=32, Hkv=8, W=128, G=32, ctx=8192, n_outliers=3, seed=2, bits=4),
    # config 4: long-context GQA-7
    "gqa7-32k": dict(L=28, B=4, Hq=28, Hkv=4, W=256, G=64, ctx=32768, n_outliers=0, seed=4, planted=True),
    # config 3: batch sweep at context 4096
    "llama3-8b-4k-b16": dict(L=32, B=16, Hq=32, Hkv=8, W=128, G=32, ctx=4096, n_outliers=3, seed=3),
    "llama3-8b-4k-b32": dict(L=16, B=32, Hq=32, Hkv=8, W=128, G=32, ctx=4096, n_outliers=3, seed=3),
    "llama3-8b-4k-b64": dict(L=8, B=64, Hq=32, Hkv=8, W=128, G=32, ctx=4096, n_outliers=3, seed=3),
    # config 5: 128k MHA (layers reduced to what is needed to exceed L2 several times)
    "mha-128k": dict(L=8, B=1, Hq=32, Hkv=32, W=256, G=32, ctx=131072, n_outliers=3, seed=5),
    # config 1 (parity-sized; latency-bound)
    "tiny": dict(L=1, B=1, Hq=8, Hkv=2, W=128, G=32, ctx=1024, n_outliers=4, seed=1),
}
D = 128
KERNELS = {"auto": 0, "scalar": 1, "mma": 2, "umma": 3}  # LQ_KERNEL_* of include/lq.h
Q_ROTATE = 16  # distinct query/new-token sets cycled through the steps


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU during the timed region (NVML)."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.005)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_min_mhz": float(min(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def reduce_max_over_ranks(values, world, device):
    """MAX over ranks of a list of per-rank timings (the job is as slow as its slowest replica)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return t.tolist()


def aggregate_throughput(units_per_rank, world, ms_max):
    """Whole-job throughput of `world` independent replicas that each processed units_per_rank."""
    return units_per_rank * world / (ms_max * 1e-3)


def make_step_inputs(wl, device, n_sets):
    """Per layer: n_sets rotating (k_new, v_new, q) triples, resident on `device`."""
    L, B, Hq, Hkv = wl["L"], wl["B"], wl["Hq"], wl["Hkv"]
    ks, vs, qs = [], [], []
    for l in range(L):
        k, v = synth.keys_values(wl["seed"] + 100, B, Hkv, n_sets, D, device, layer=l,
                                 outliers=wl.get("_outliers"))
        ks.append([k[:, :, i:i + 1].contiguous() for i in range(n_sets)])
        vs.append([v[:, :, i:i + 1].contiguous() for i in range(n_sets)])
        qs.append([synth.queries(wl["seed"], B, Hq, D, i, device, layer=l) for i in range(n_sets)])
    return ks, vs, qs


def prefill(cache, wl, device, layers=None, chunk=None, sink=None):
    """Append ctx tokens to every layer, generated on `device`: the whole prompt in one call (one
    ingestion launch per layer) when K and V of a layer fit in 4 GB, else 1024 tokens at a time.
    sink(layer, k, v) additionally receives each chunk (used to feed the CPU oracle)."""
    L, B, Hkv, ctx = wl["L"], wl["B"], wl["Hkv"], wl["ctx"]
    if chunk is None:
        chunk = ctx if 2 * B * Hkv * ctx * D * 2 <= 4e9 else 1024
    u = synth.unit_vectors(wl["seed"], Hkv, D) if wl.get("planted") else None
    for l in (range(L) if layers is None else layers):
        for t0 in range(0, ctx, chunk):
            n = min(chunk, ctx - t0)
            k, v = synth.keys_values(wl["seed"], B, Hkv, n, D, device, token_start=t0, token_total=ctx,
                                     outliers=wl.get("_outliers"), layer=l)
            if u is not None:
                k = synth.plant_spikes(k, u, 16.0, t0, ctx)
            if cache is not None:
                cache.append(l, k, v)
            if sink is not None:
                sink(l, k, v)


def run_ours(args, wl, rank, world, device):
    from paper_2503_19950_b200 import LogQuantCache, build
    build.build()
    L, B, Hq, Hkv, W, G, ctx = (wl[k] for k in ("L", "B", "Hq", "Hkv", "W", "G", "ctx"))
    steps, warmup = args.steps, args.warmup
    total_steps = 2 * (steps + warmup) + steps + warmup + 8  # device-timed, profiled and host-buffer passes
    bits = wl.get("bits", 2)
    cache = LogQuantCache(L, B, Hq, Hkv, W, G, max_tokens=ctx + total_steps + 8, device=device.index or 0, bits=bits,
                          n_splits=args.n_splits, kernel=KERNELS[args.kernel], flags=0 if args.no_overlap else 1)
    pad = wl.get("pad")
    n_pad = sum(pad) if pad else 0
    if pad:
        cache.set_padding(pad)
    prefill(cache, wl, device)
    ks, vs, qs = make_step_inputs(wl, device, Q_ROTATE)
    outs = [torch.empty(B, Hq, D, device=device) for _ in range(L)]
    torch.cuda.synchronize()

    def one_step(i):
        s = i % Q_ROTATE
        for l in range(L):
            cache.append_decode_attn(l, ks[l][s], vs[l][s], qs[l][s], outs[l])

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    def timed(n, fn, start_idx):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        kv_tokens = 0
        barrier()
        ev0.record()
        for i in range(n):
            fn(start_idx + i)
            inf = cache.info_fast()
            kv_tokens += (B * (inf[0] + inf[1]) - n_pad) * L
        ev1.record()
        barrier()
        return ev0.elapsed_time(ev1), kv_tokens

    step_idx = 0
    for i in range(warmup):
        one_step(step_idx)
        step_idx += 1
    launches0 = cache.info(0).n_kernel_launches
    with ClockSampler(device.index or 0) as clk:
        ms, kv_tokens = timed(steps, one_step, step_idx)
    step_idx += steps
    launches = cache.info(0).n_kernel_launches - launches0
    bytes_step_last = sum(cache.info(l).bytes_decode_step for l in range(L))

    # ---- kernel-only timing of the split-K attention kernel (roofline) ----
    # (a) the kernel launched back to back, rotating over the L layer caches (more than L2 between two
    #     visits of a cache), CUDA events around every round of L launches: median round / L;
    # (b) every launch of a step bracketed by its own pair of events (includes the event and launch gap).
    # The kernel runs the board at its power limit: after about 0.1 s of back-to-back launches `sw_power_cap` sets
    # in and the SM clock drops by 4 - 10 %.  The peak in the denominator is a burst figure (best of 10 copies), so
    # the rounds are taken the same way, after a pause that lets the board settle; the figure after 0.5 s of
    # continuous launches is reported beside it (`sustained`), with the clocks seen during that leg.
    def timed_rounds(n):
        evs = []
        for rep in range(n):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for p in range(passes):
                s = (step_idx + rep + p) % Q_ROTATE
                for l in range(L):
                    cache.decode_attn(l, qs[l][s], outs[l])
            e1.record()
            evs.append((e0, e1))
        torch.cuda.synchronize()
        return [e0.elapsed_time(e1) * 1e3 / passes for e0, e1 in evs]

    passes = max(1, 32 // L)  # at least 32 launches between two event records: a record serialises its neighbours
    torch.cuda.synchronize()
    time.sleep(1.0)
    round_us = sorted(timed_rounds(max(8, min(steps, 64)) + 3)[3:])
    b2b_us = round_us[len(round_us) // 2] / L
    b2b_best_us = round_us[0] / L
    bytes_b2b = sum(cache.info(l).bytes_decode_step for l in range(L)) / L
    sustained = None
    if steps >= 32:
        n_sus = int(0.6e6 / max(b2b_us * L * passes, 1.0)) + 1
        with ClockSampler(device.index or 0) as clk_sus:
            sus = timed_rounds(n_sus)
        tail = sorted(sus[-max(8, n_sus // 6):])
        sustained = {"us_per_launch": tail[len(tail) // 2] / L, "rounds": n_sus, "seconds": sum(sus) * 1e-6,
                     "what": "median of the last sixth of %d rounds launched back to back without a pause" % n_sus,
                     "clocks": clk_sus.summary()}
    if pad:
        # algorithmic bytes of a padded batch: the stored bytes of the tokens that are not padding
        img, inf0 = cache.export(0), cache.info(0)
        real_q = sum(int((img["quant_ids"] >= pb).sum()) for pb in pad)
        real_f = sum(int((img["kept_ids"] >= pb).sum()) for pb in pad)
        bytes_b2b = Hkv * (real_q * inf0.bytes_quant_per_token + real_f * 4 * D)
        del img
    cache.profile_enable(True)
    byte_sum = 0
    for i in range(min(steps, 8192 // L)):
        s = (step_idx + i) % Q_ROTATE
        for l in range(L):
            cache.append(l, ks[l][s], vs[l][s])
            byte_sum += cache.info(l).bytes_decode_step
            cache.decode_attn(l, qs[l][s], outs[l])
    k_ms, k_n = cache.profile_read()
    cache.profile_enable(False)
    step_idx += min(steps, 8192 // L)

    # ---- end to end through the C-ABI with host buffers (pinned), copies inside the timed region ----
    hk = [[ks[l][s].cpu().pin_memory() for s in range(Q_ROTATE)] for l in range(L)]
    hv = [[vs[l][s].cpu().pin_memory() for s in range(Q_ROTATE)] for l in range(L)]
    hq = [[qs[l][s].cpu().pin_memory() for s in range(Q_ROTATE)] for l in range(L)]
    hout = [torch.empty(B, Hq, D, dtype=torch.float32).pin_memory() for _ in range(L)]

    def host_step(i):
        s = i % Q_ROTATE
        for l in range(L):
            cache.decode_step_host(l, hk[l][s], hv[l][s], hq[l][s], hout[l], sync=False)
        torch.cuda.current_stream().synchronize()  # the step's result is on the host

    e2e_steps = max(3, min(steps, 32))
    for i in range(3):
        host_step(step_idx)
        step_idx += 1
    t0 = time.perf_counter()
    barrier()
    t0 = time.perf_counter()
    kv_e2e = 0
    for i in range(e2e_steps):
        host_step(step_idx + i)
        inf = cache.info_fast()
        kv_e2e += (B * (inf[0] + inf[1]) - n_pad) * L
    barrier()
    e2e_s = time.perf_counter() - t0
    # ---- one window-overflow event over all layers at once (lq_compress(layer=-1)) ----
    comp = None
    try:
        ccache = LogQuantCache(L, B, Hq, Hkv, W, G, max_tokens=8 * W, device=device.index or 0, auto_compress=False,
                               bits=bits)
        kf, vf = synth.keys_values(wl["seed"] + 7, B, Hkv, 3 * W, D, device, outliers=wl.get("_outliers"))
        k1, v1 = kf[:, :, :W].contiguous(), vf[:, :, :W].contiguous()
        evs = []
        for rep in range(6):
            for l in range(L):
                ccache.append(l, kf, vf) if rep == 0 else ccache.append(l, k1, v1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            ccache.compress(-1)
            e1.record()
            torch.cuda.synchronize()
            evs.append(e0.elapsed_time(e1) * 1e3)
        us = float(np.median(evs[1:]))
        rd = L * B * Hkv * (2 * W * 256 + W * 512)          # removed rows + back-fill sources, K and V
        wr = L * B * Hkv * (W * (1024 // G + 32 * bits) + W * 512)   # packed tiles + back-filled rows
        comp = {"us_per_event": us, "layers": L, "tokens_per_s": L * B * W / (us * 1e-6),
                "gbs": (rd + wr) / (us * 1e-6) / 1e9, "read_bytes": rd, "write_bytes": wr}
        ccache.close()
    except Exception as exc:  # the main numbers stand without it
        comp = {"error": str(exc)}
    planted_bf16 = None
    if wl.get("planted"):
        # context only: which of the planted high-logit tokens (distances 2^i behind the end of the prompt) are
        # still at full precision in the log-spaced selection at the end of the run
        kept = set(int(t) for t in cache.export(0)["kept_ids"])
        planted_bf16 = [1 << i for i in range(32) if (1 << i) <= ctx and (ctx - (1 << i)) in kept]
    status = cache.kernel_status()
    assert status == 0, f"kernel status word {status}"
    assert all(torch.isfinite(o).all() for o in outs)

    ms_max, e2e_ms_max = reduce_max_over_ranks([ms, e2e_s * 1e3], world, device)
    peak, peak_kind = peaks()
    bytes_per_launch = bytes_b2b
    achieved = bytes_per_launch / (b2b_us * 1e-6) / 1e9
    isolated_us = k_ms / max(k_n, 1) * 1e3 if k_n else None
    inf = cache.info(0)
    line = {
        "metric": "decode_attn_kv_tokens_per_s", "value": aggregate_throughput(kv_tokens, world, ms_max),
        "unit": "KV tokens/s", "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_max / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "layers": L, "batch": B, "q_heads": Hq, "kv_heads": Hkv,
                   "head_dim": D, "context": ctx, "window": W, "group": G, "bits": bits,
                   "padding": pad, "planted_distances_still_bf16": planted_bf16, "n_quant": int(inf.n_quant), "n_fp": int(inf.n_fp), "n_splits": int(inf.n_splits), "n_ctas": int(inf.n_ctas),
                   "step": "per layer: lq_append_decode_attn (append and attention in one launch; the overflow step and "
                           "a separate append when the window is full)",
                   "l2": "inputs larger than L2: %.2f GB of cache touched per step" % (bytes_step_last / 1e9),
                   "merge": ("partials summed on arrival with global atomics (more than 12 CTAs per (b, kv) pair; not "
                             "bit-reproducible), records as fallback" if int(inf.n_splits) >= 12 else
                             "ordered merge of the CTA records by the last CTA of a pair (bit-reproducible)"),
                   "n_ctas_overlapped": int(getattr(inf, "n_ctas_overlapped", 0)),
                   "launch_overlap": ("every launch waits for the one before it" if args.no_overlap else
                                      "LQ_FLAG_OVERLAP_DECODE: attention launches of consecutive layers overlap (a launch streams its "
                                      "own layer's stores while the previous one merges, and waits for it before the shared "
                                      "workspace); roofline.serialized is the same kernel without it"),
                   "replicas": "independent per GPU, no collective on the data path"},
        "per_layer_us": ms_max / steps / L * 1e3,
        "algorithmic_gbs_whole_step": bytes_step_last / (ms_max / steps * 1e-3) / 1e9,
        "gpu_launches": int(launches),
        # bf16 cache bytes / mixed cache bytes actually read per step (scale and zero counted)
        "compression_ratio": (B * Hkv * (int(inf.n_quant) + int(inf.n_fp)) * 4 * D) / max(int(inf.bytes_decode_step), 1),
        # the paper's own formula (Eq. 4-5), which counts the 2-bit codes only: 16 L / (2 (L - R) + 16 R) with L tokens
        # in the cache and R of them at full precision (for bits = 4: 4 in place of 2)
        "compression_ratio_paper_formula": 16.0 * (int(inf.n_quant) + int(inf.n_fp)) /
                                           (bits * int(inf.n_quant) + 16.0 * int(inf.n_fp)),
        "compress_event": comp,
        "clocks": clk.summary(),
        "e2e": {"value": aggregate_throughput(kv_e2e, world, e2e_ms_max), "unit": "KV tokens/s",
                "h2d_bytes_per_step": L * (2 * B * Hkv * D * 2 + B * Hq * D * 2),
                "d2h_bytes_per_step": L * B * Hq * D * 4, "steps": e2e_steps,
                "api": "lq_decode_step_host (pinned host buffers, one stream sync per step)"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": None, "peak_kind": peak_kind,
                     "kernel": "lq_decode_umma_kernel" if args.kernel == "umma" else "lq_decode_mma_kernel", "bytes_per_launch": bytes_per_launch,
                     "us_per_launch": b2b_us, "us_per_launch_best": b2b_best_us,
                     "sustained": None if sustained is None else dict(
                         sustained, achieved=bytes_b2b / (sustained["us_per_launch"] * 1e-6) / 1e9,
                         frac=bytes_b2b / (sustained["us_per_launch"] * 1e-6) / 1e9 / peak),
                     "us_per_launch_quartiles": [round(round_us[int(f * (len(round_us) - 1))] / L, 3) for f in (0, 0.25, 0.5, 0.75, 1)],
                     "timing": "median over %d rounds of %d back-to-back launches (%d passes over %d layer caches), taken "
                               "after a 1 s pause (burst, like the peak); `sustained`: after 0.6 s without a pause" % (
                         len(round_us), passes * L, passes, L),
                     "us_per_launch_isolated": isolated_us,
                     "frac_isolated": (byte_sum / max(k_n, 1)) / (isolated_us * 1e-6) / 1e9 / peak if isolated_us else None,
                     "launches_timed": len(round_us) * L * passes,
                     "frac_of_8tbs_nominal": achieved / 8000.0},
    }
    # DRAM bytes per launch of the dominant kernel, from the committed ncu summary of this workload
    traffic_file = os.path.join(ROOT, "profiles", "decode_attention_%s.md" % args.workload)
    if os.path.exists(traffic_file):
        import re
        with open(traffic_file) as f:
            m = re.search(r"dram_bytes_per_launch:\s*([0-9.eE+]+)", f.read())
        if m:
            line["roofline"]["traffic"] = float(m.group(1))
    line["_replay"] = {"ks0": ks[0], "vs0": vs[0], "qs0": qs[0], "n_decode_tokens": int(cache.info(0).n_seen) - ctx}
    return line, cache


def roofline_only(name, device, layers, rounds=24, n_splits=0, kernel=0, flags=1):
    """Back-to-back timing of the attention kernel on another workload (a few layer caches, a few seconds):
    the same measurement as the `roofline` object of the main line."""
    from paper_2503_19950_b200 import LogQuantCache
    wl = dict(WORKLOADS[name], L=layers)
    wl["_outliers"] = synth.outlier_channels(wl["seed"], wl["Hkv"], D, wl["n_outliers"]) if wl["n_outliers"] else None
    L, B, Hq, Hkv, W, G, ctx = (wl[k] for k in ("L", "B", "Hq", "Hkv", "W", "G", "ctx"))
    cache = LogQuantCache(L, B, Hq, Hkv, W, G, max_tokens=ctx + 64, device=device.index or 0, bits=wl.get("bits", 2),
                          n_splits=n_splits, kernel=kernel, flags=flags)
    prefill(cache, wl, device)
    ks, vs, qs = make_step_inputs(wl, device, 4)
    outs = [torch.empty(B, Hq, D, device=device) for _ in range(L)]
    for l in range(L):  # first decode step: the overflow step runs here, the timed launches see the state after it
        cache.append_decode_attn(l, ks[l][0], vs[l][0], qs[l][0], outs[l])
    evs = []
    passes = max(1, 32 // L)  # launches between two event records: as many as the main workload's 32 layers
    torch.cuda.synchronize()
    time.sleep(1.0)  # burst figure, like the peak it is divided by (see the main workload's rounds)
    for rep in range(rounds + 3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for p in range(passes):
            for l in range(L):
                cache.decode_attn(l, qs[l][(rep + p) % 4], outs[l])
        e1.record()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    us = sorted(e0.elapsed_time(e1) * 1e3 / passes for e0, e1 in evs[3:])
    b2b_us = us[len(us) // 2] / L
    inf = cache.info(0)
    nbytes = int(inf.bytes_decode_step)
    peak, peak_kind = peaks()
    ok = cache.kernel_status() == 0 and all(bool(torch.isfinite(o).all()) for o in outs)
    cache.close()
    return {"workload": name, "layers": L, "bound": "hbm", "achieved": nbytes / (b2b_us * 1e-6) / 1e9, "peak": peak,
            "unit": "GB/s", "frac": nbytes / (b2b_us * 1e-6) / 1e9 / peak, "peak_kind": peak_kind,
            "bytes_per_launch": nbytes, "us_per_launch": b2b_us, "us_per_launch_best": us[0] / L,
            "kv_tokens_per_s": B * (int(inf.n_quant) + int(inf.n_fp)) / (b2b_us * 1e-6),
            "n_quant": int(inf.n_quant), "n_fp": int(inf.n_fp), "n_ctas": int(inf.n_ctas), "finite_and_status_ok": ok,
            "frac_of_8tbs_nominal": nbytes / (b2b_us * 1e-6) / 1e9 / 8000.0,
            "timing": "median over %d rounds of %d back-to-back launches (%d passes over %d layer caches)" % (
                len(us), passes * L, passes, L)}


def parity_against_oracle(cache, wl, device, replay):
    """Checker leg (uses oracle/): replays every token layer 0 of the timed cache has received into the CPU oracle,
    takes one more decode step through the call the bench times (lq_append_decode_attn) and compares the canonical
    image and the attention output of that step with the oracle's."""
    import oracle
    B, Hq, Hkv, W, G = (wl[k] for k in ("B", "Hq", "Hkv", "W", "G"))
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G, bits=wl.get("bits", 2))
    prefill(None, dict(wl, L=1), device, sink=lambda l, k, v: oc.append(synth.bf16_bits(k), synth.bf16_bits(v)))
    n = replay["n_decode_tokens"]
    for j in range(n + 1):  # decode token j of a layer was set j % Q_ROTATE; the last one is appended below
        s = j % Q_ROTATE
        oc.append(synth.bf16_bits(replay["ks0"][s]), synth.bf16_bits(replay["vs0"][s]))
    s = n % Q_ROTATE
    out = torch.full((B, Hq, D), float("nan"), device=device)
    cache.append_decode_attn(0, replay["ks0"][s], replay["vs0"][s], replay["qs0"][s], out)
    torch.cuda.synchronize()
    inf = cache.info(0)
    state_ok = (inf.n_seen, inf.n_fp, inf.n_quant, inf.n_events) == (oc.n_seen, oc.n_fp, oc.n_quant, oc.n_events)
    got, want = cache.export(0), oc.export()
    image_ok = state_ok and all(np.array_equal(got[key], want[key]) for key in want)
    pad = wl.get("pad")
    if pad:
        ref = oc.attention_subset(synth.bf16_bits(replay["qs0"][s]), 1.0 / np.sqrt(D), pad=pad)
    else:
        ref = oc.attention(synth.bf16_bits(replay["qs0"][s]), 1.0 / np.sqrt(D), n_threads=os.cpu_count() or 1)
    o = out.cpu().numpy().astype(np.float64)
    err = float(np.abs(o - ref).max()) if np.isfinite(o).all() else float("inf")
    tol = 2e-3 * float(np.abs(ref).max()) + 1e-3
    return {"max_err": err, "tol": tol, "image_bit_exact": bool(image_ok), "ok": bool(image_ok and err <= tol),
            "checked": "layer 0 after %d decode tokens, one step through lq_append_decode_attn: canonical image and "
                       "[B, Hq, D] output against the float64 oracle" % (n + 1)}


def oracle_compress_event(wl, device, reps=5):
    """Times the CPU oracle on one window-overflow step of one layer (the append that finds 3W tokens)."""
    import oracle
    B, Hq, Hkv, W, G = (wl[k] for k in ("B", "Hq", "Hkv", "W", "G"))
    kf, vf = synth.keys_values(wl["seed"] + 7, B, Hkv, 3 * W + 1, D, device, outliers=wl.get("_outliers"))
    kb, vb = synth.bf16_bits(kf), synth.bf16_bits(vf)
    ts = []
    for rep in range(reps):
        oc = oracle.OracleCache(B, Hq, Hkv, D, W, G, bits=wl.get("bits", 2))
        oc.append(np.ascontiguousarray(kb[:, :, :3 * W]), np.ascontiguousarray(vb[:, :, :3 * W]))
        k1, v1 = np.ascontiguousarray(kb[:, :, 3 * W:]), np.ascontiguousarray(vb[:, :, 3 * W:])
        t0 = time.perf_counter()
        oc.append(k1, v1)
        ts.append(time.perf_counter() - t0)
        assert oc.n_events == 1
        oc.close()
    us = float(np.median(ts)) * 1e6
    return {"us_per_event_one_layer": us, "tokens_per_s": B * W / (us * 1e-6), "threads": 1,
            "what": "oracle append of the token that finds 3W full-precision tokens: filter, quantise and pack W tokens "
                    "of all %d sequences, one layer" % B}


def oracle_layer_step(wl, device, n_threads, min_seconds, max_reps, warmup=0):
    """Times the CPU oracle on one layer of the workload: append one token + attention.
    Runs until min_seconds of timed work or max_reps steps, whichever comes first (at least one)."""
    import oracle
    B, Hq, Hkv, W, G, ctx = (wl[k] for k in ("B", "Hq", "Hkv", "W", "G", "ctx"))
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G, bits=wl.get("bits", 2))
    wl1 = dict(wl, L=1)
    prefill(None, wl1, device, sink=lambda l, k, v: oc.append(synth.bf16_bits(k), synth.bf16_bits(v)))
    k, v = synth.keys_values(wl["seed"] + 100, B, Hkv, Q_ROTATE, D, device, layer=0, outliers=wl.get("_outliers"))
    kb, vb = synth.bf16_bits(k), synth.bf16_bits(v)
    reps, t_total, kv = 0, 0.0, 0
    times = []
    for i in range(warmup):
        q = synth.bf16_bits(synth.queries(wl["seed"], B, Hq, D, i % Q_ROTATE, device, layer=0))
        oc.append(np.ascontiguousarray(kb[:, :, i % Q_ROTATE:i % Q_ROTATE + 1]),
                  np.ascontiguousarray(vb[:, :, i % Q_ROTATE:i % Q_ROTATE + 1]))
        oc.attention(q, 1.0 / np.sqrt(D), n_threads=n_threads)
    while (t_total < min_seconds and reps < max_reps) or reps < 1:
        s = reps % Q_ROTATE
        q = synth.bf16_bits(synth.queries(wl["seed"], B, Hq, D, s, device, layer=0))
        t0 = time.perf_counter()
        oc.append(np.ascontiguousarray(kb[:, :, s:s + 1]), np.ascontiguousarray(vb[:, :, s:s + 1]))
        if wl.get("pad"):
            oc.attention_subset(q, 1.0 / np.sqrt(D), pad=wl["pad"])  # (single-threaded in the oracle)
        else:
            oc.attention(q, 1.0 / np.sqrt(D), n_threads=n_threads)
        dt = time.perf_counter() - t0
        times.append(dt)
        t_total += dt
        kv += B * (oc.n_quant + oc.n_fp) - sum(wl.get("pad") or [])
        reps += 1
    return kv / t_total, reps, t_total, times


def spawn_replicas(n, argv, need_gpus=True, timeout=None):
    """Re-runs this script as n ranks under torch.distributed.run (rendezvous on 127.0.0.1).  Fails loudly when
    the machine has fewer than n GPUs."""
    import socket
    import subprocess
    if need_gpus and torch.cuda.device_count() < n:
        sys.stderr.write("bench.py: --gpus %d asked for, %d CUDA device(s) visible\n" % (n, torch.cuda.device_count()))
        return 2
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.run(cmd, timeout=timeout).returncode


def replica_selftest(args, rank, world):
    """CPU-only check of the replica plumbing (no kernel, no oracle): every rank 'processes' a fixed number of
    units in a rank-dependent time; rank 0 prints the line the real run would print from these."""
    torch.distributed.init_process_group("gloo")
    units, ms = 1000, 10.0 + 5.0 * rank
    ms_max = reduce_max_over_ranks([ms], world, torch.device("cpu"))[0]
    if rank == 0:
        print(json.dumps({"impl": "replica-selftest", "n_gpus": world, "value": aggregate_throughput(units, world, ms_max),
                          "ms_per_step": ms_max, "scaling": "weak"}))
    torch.distributed.barrier()
    torch.distributed.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "replica-selftest"])
    ap.add_argument("--workload", default="llama3-8b-8k", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="override the number of stacked layer caches (profiling runs)")
    ap.add_argument("--n-splits", type=int, default=0, help="split-K CTAs per (batch row, KV head); 0 = library default")
    ap.add_argument("--shorten-prefill", type=int, default=0,
                    help="prefill this many tokens fewer than the workload's context (e.g. W/2: the overflow step then "
                         "falls in the middle of the timed steps instead of on the first decode step)")
    ap.add_argument("--kernel", default="auto", choices=sorted(KERNELS), help="decode-attention kernel (LQ_KERNEL_*)")
    ap.add_argument("--no-overlap", action="store_true",
                    help="create the caches without LQ_FLAG_OVERLAP_DECODE: every attention launch waits for the one before it")
    ap.add_argument("--also", default=None,
                    help="comma-separated workloads whose attention kernel is timed back to back as well and reported "
                         "under roofline_<workload> (default: the other configurations -- gqa7-32k, the batch sweep, mha-128k -- beside the default workload)")
    ap.add_argument("--also-layers", type=int, default=32, help="layer caches of the --also workloads")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.also is None:
        args.also = ("gqa7-32k,llama3-8b-4k-b16,llama3-8b-4k-b32,llama3-8b-4k-b64,mha-128k"
                     if args.workload == "llama3-8b-8k" and args.layers == 0 else "")

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # replicas only: --gpus N without a launcher starts N ranks of this script (one per GPU), which time N
        # independent replicas; no collective touches the data path
        return spawn_replicas(args.gpus, sys.argv[1:], need_gpus=args.impl == "ours")

    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    wl = dict(WORKLOADS[args.workload])
    if args.layers > 0:
        wl["L"] = args.layers
    if args.shorten_prefill > 0:
        wl["ctx"] = max(1, wl["ctx"] - args.shorten_prefill)
    wl["_outliers"] = synth.outlier_channels(wl["seed"], wl["Hkv"], D, wl["n_outliers"]) if wl["n_outliers"] else None
    cores = os.cpu_count() or 1

    if args.impl == "replica-selftest":
        return replica_selftest(args, rank, world)
    if args.impl == "reference":
        if rank != 0:
            return 0
        import oracle
        oracle.build()
        device = torch.device("cuda", local) if torch.cuda.is_available() else torch.device("cpu")
        tput, reps, t_total, times = oracle_layer_step(wl, device, cores, min_seconds=1e9, max_reps=max(args.steps, 1),
                                                       warmup=max(args.warmup, 0))
        sample = "one of %d layers of %s per step: append 1 token + attention, float64" % (wl["L"], args.workload)
        line = {"impl": "reference", "metric": "decode_attn_kv_tokens_per_s", "value": tput, "unit": "KV tokens/s",
                "n_gpus": args.gpus, "steps": reps, "warmup": args.warmup, "ms_per_step": t_total / reps * 1e3,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": {"workload": args.workload, "batch": wl["B"], "q_heads": wl["Hq"], "kv_heads": wl["Hkv"],
                           "context": wl["ctx"], "window": wl["W"], "group": wl["G"]},
                "cpu_baseline": {"value": tput, "unit": "KV tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
                "e2e": {"value": tput, "unit": "KV tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return 0

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the LogQuant kernels")
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=device)
    line, cache = run_ours(args, wl, rank, world, device)
    replay = line.pop("_replay")
    parity_failed = False
    if rank == 0:
        for name in [n for n in args.also.split(",") if n]:
            try:
                line["roofline_" + name.replace("-", "_")] = roofline_only(name, device, args.also_layers,
                                                                           kernel=KERNELS[args.kernel],
                                                                           flags=0 if args.no_overlap else 1)
            except Exception as exc:  # the main line stands without it
                line["roofline_" + name.replace("-", "_")] = {"error": str(exc)}
        if not args.no_overlap:
            # the same kernel with every launch waiting for the one before it (LQ_FLAG_OVERLAP_DECODE off)
            try:
                ser = roofline_only(args.workload, device, max(8, args.also_layers), kernel=KERNELS[args.kernel], flags=0)
                line["roofline"]["serialized"] = {k: ser[k] for k in ("us_per_launch", "achieved", "frac", "layers")}
            except Exception as exc:
                line["roofline"]["serialized"] = {"error": str(exc)}
        if not args.no_cpu_baseline:
            import oracle
            oracle.build()
            line["parity"] = parity_against_oracle(cache, wl, device, replay)
            parity_failed = not line["parity"]["ok"]
            if isinstance(line.get("compress_event"), dict) and "error" not in line["compress_event"]:
                line["compress_event"]["cpu_oracle"] = oracle_compress_event(wl, device)
            tput, reps, t_total, _ = oracle_layer_step(wl, device, cores, min_seconds=10.0, max_reps=512)
            tput1, reps1, t1, _ = oracle_layer_step(wl, device, 1, min_seconds=3.0, max_reps=64)
            line["cpu_baseline"] = {"value": tput, "unit": "KV tokens/s", "cores": cores, "kind": "oracle",
                                    "sample": "%d decode steps of one of the %d layers (append 1 token + float64 "
                                              "attention over all %d sequences), %.1f s" % (reps, wl["L"], wl["B"], t_total),
                                    "single_thread": {"value": tput1, "steps": reps1, "seconds": t1},
                                    "hardware_concurrency": oracle.hardware_threads(),
                                    "paper_context": "the paper reports +25 % throughput and +60 % batch size over a bf16 "
                                                     "cache on an H100 through the HuggingFace pipeline (Sec. 3.2.4): "
                                                     "end-to-end generation, another machine; context only"}
        print(json.dumps(line))
    cache.close()
    if world > 1:
        torch.distributed.barrier()
        torch.distributed.destroy_process_group()
    if parity_failed:
        sys.stderr.write("bench.py: the timed path disagrees with the oracle: %s\n" % json.dumps(line["parity"]))
        return 1
    return 0


if __name__ == "__main__":
    sys.exit(main())
