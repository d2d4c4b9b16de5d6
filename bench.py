#!/usr/bin/env python
"""Benchmark of the compressed-cache decode hot path on B200.

Workload (N = 1): Llama3-8B-shaped single-layer decode, B=4 sequences, 32 query heads, 8 KV heads,
d_h=128, T=32768 tokens of context per sequence, r_k=r_v=64, bf16 compressed cache in 64-token pages
handed out from a shuffled pool.  Keys are a rank-48 Gaussian signal plus 0.1 N(0,1) noise, values and
queries Gaussian, bases from seeded QR -- all synthetic.

A step = one decode step of one layer: project and append the new token's k, v into the cache, project the
queries, split-T attention over the T+1 cached tokens in the compressed space, merge the chunks and
back-project (every kernel of the path).  The cache itself is built once, before timing, by the library's
own prefill-compression kernel, which is timed separately and reported under "prefill".  Steps rotate over
several independent layer caches, each larger than L2, so no step finds its cache in L2.

metric  = effective HBM bandwidth over the compressed cache bytes a step must read
          (B * Hkv * (T+1) * 2 * (r_k + r_v) bytes per step); tokens/s is reported next to it.
Prints one JSON line.  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

SEED = 0
CFG2 = dict(B=4, Hq=32, Hkv=8, T=32768, r_k=64, r_v=64)
# single-layer decode workloads that share the config-2 harness (the headline line is config 2)
SINGLE_LAYER = {
    "config2": dict(CFG2, name="config2: Llama3-8B-shaped single-layer decode, B=4 Hq=32 Hkv=8 d=128 T=32768 r_k=r_v=64"),
    "config4a": dict(B=1, Hq=32, Hkv=8, T=131072, r_k=48, r_v=64,
                     name="config4a: one long sequence, B=1 Hq=32 Hkv=8 d=128 T=131072 r_k=48 r_v=64"),
    "config4b": dict(B=16, Hq=32, Hkv=8, T=16384, r_k=64, r_v=64, ragged=True,
                     name="config4b: ragged batch, B=16 Hq=32 Hkv=8 d=128 lengths uniform in [1024,16384] r_k=r_v=64"),
}
N_CACHES = 4               # rotating layer caches (each 256 MiB of compressed rows)
# DRAM bytes (read + write) of one launch of decode_persistent_kernel<64,64> on config 2, from the ncu capture whose summary
# is the named file (mean of its two launches).  It describes the kernel AS CAPTURED: set both to None whenever
# csrc/stief_decode.cuh or csrc/stief_partition.cuh changes, until the capture has been retaken (--traffic overrides).
CAPTURED_TRAFFIC = 273.58e6
CAPTURED_TRAFFIC_SOURCE = "profiles/decode_persistent_kernel_config2.md (ncu --set full capture of this kernel, mean of two launches)"
METRIC = "decode_attn_effective_hbm_gbs"
UNIT = "GB/s"


def seq_lengths(cfg):
    from paper_2601_21686_b200 import inputs as I
    if cfg.get("ragged"):
        return [int(x) for x in I.ragged_lengths(SEED, cfg["B"])]
    return [cfg["T"]] * cfg["B"]


def step_bytes(cfg) -> int:
    """Compressed-cache bytes one decode step must read: every cached row of every KV head, new token included."""
    return sum(n + 1 for n in seq_lengths(cfg)) * cfg["Hkv"] * 2 * (cfg["r_k"] + cfg["r_v"])


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d["hbm_gbs"]), float(d.get("bf16_tflops", 1590.0)), "measured"
        except Exception:
            pass
    return 6650.0, 1590.0, "fallback"


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50",
                                          "-i", str(self.idx)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()

    def summary(self, t0: float, t1: float):
        sm, mx, reasons = [], [], set()
        for ts, line in self.rows:
            if ts < t0 - 0.05 or ts > t1 + 0.15:
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# the CUDA arm
# ------------------------------------------------------------------------------------------------
def build_caches(cfg, n_caches, dev, S, I):
    """n_caches independent layer caches, filled by the library's prefill kernel from seeded K, V."""
    B, Hq, Hkv, T, r_k, r_v = (cfg[k] for k in ("B", "Hq", "Hkv", "T", "r_k", "r_v"))
    lens = seq_lengths(cfg)
    T = max(lens)
    pg = I.make_paging(SEED, lens, reserve_tokens=1)
    bt = torch.from_numpy(pg.block_table).to(dev)
    lens = torch.from_numpy(pg.seq_lens).to(dev)
    batch = S.Batch(bt, lens)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    layers, inputs = [], []
    for l in range(n_caches):
        U_k, U_v = I.stiefel_bases(SEED, l, Hkv, r_k, r_v)
        layer = S.Layer(Hq, Hkv, r_k, r_v, U_k.to(dev), U_v.to(dev),
                        torch.zeros(pg.num_pages, Hkv, 64, r_k, dtype=torch.bfloat16, device=dev),
                        torch.zeros(pg.num_pages, Hkv, 64, r_v, dtype=torch.bfloat16, device=dev))
        K = I.lowrank_keys(SEED, l, B, T, Hkv, device=dev)
        V = I.gaussian_kv(SEED, I.TAG_V, l, B, T, Hkv, device=dev)
        S.stief_prefill_compress(layer, batch, K, V, status=status)      # the real fill (and a warm-up)
        layers.append(layer)
        inputs.append((K, V))
    torch.cuda.synchronize()
    # timed: the per-layer launches of one prompt back to back (different inputs and pools per layer, each layer's
    # inputs larger than L2), overlapped the way a 32-layer prefill would launch them
    reps = 3
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for r in range(reps):
        for l in range(n_caches):
            S.stief_prefill_compress(layers[l], batch, inputs[l][0], inputs[l][1], status=status,
                                     flags=S.STIEF_PREFILL_OVERLAP_PREVIOUS if (r or l) else 0)
    e1.record()
    torch.cuda.synchronize()
    prefill_ms = [e0.elapsed_time(e1) / (reps * n_caches)]
    del inputs
    assert int(status.item()) == 0, f"device status {int(status.item())} while building the cache"
    return layers, batch, status, prefill_ms


def run_ours(args):
    import paper_2601_21686_b200 as S
    from paper_2601_21686_b200 import inputs as I
    from paper_2601_21686_b200 import build as Bld

    from paper_2601_21686_b200 import replicas as R
    me = R.replica_from_env()
    world, rank, local_rank = me.world, me.rank, me.local_rank
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    R.init(me, "nccl", dev)
    if rank == 0:
        Bld.build()
    R.barrier(me)
    S.lib()

    cfg = dict(SINGLE_LAYER[args.workload])
    if args.ranks:                                   # a variant of the workload at other ranks (not the headline)
        cfg["r_k"], cfg["r_v"] = (int(x) for x in args.ranks.split(","))
        cfg["name"] += f" [ranks overridden: r_k={cfg['r_k']} r_v={cfg['r_v']}]"
    n_caches = args.caches
    B, Hq, Hkv, T, r_k, r_v = (cfg[k] for k in ("B", "Hq", "Hkv", "T", "r_k", "r_v"))
    layers, batch, status, prefill_ms = build_caches(cfg, n_caches, dev, S, I)
    ns = args.num_parts or S.stief_decode_num_parts()
    ws = torch.empty(S.stief_decode_workspace_bytes(B, Hq, Hkv, r_v, ns) // 4, dtype=torch.float32, device=dev)
    S.stief_decode_workspace_init(ws)
    out = torch.empty(B, Hq, 128, dtype=torch.bfloat16, device=dev)
    n_in = 8
    qs = [I.queries(SEED, 0, B, Hq, scale=1.0 / np.sqrt(128.0), device=dev, step=i) for i in range(n_in)]
    kvs = [I.new_token_kv(SEED, 0, B, Hkv, device=dev, step=i) for i in range(n_in)]

    # Consecutive steps work on different layer caches and their inputs are resident before the loop, which
    # is what STIEF_DECODE_OVERLAP_PREVIOUS asks for: each launch may take over SMs as the previous one drains.
    overlap = S.STIEF_DECODE_OVERLAP_PREVIOUS if (args.overlap and n_caches >= 2) else 0

    def step(i, flags=overlap):
        S.stief_decode_step(layers[i % n_caches], batch, qs[i % n_in], kvs[i % n_in][0], kvs[i % n_in][1], ws, out,
                            num_parts=ns, status=status, flags=flags)

    def barrier():
        R.barrier(me)
        torch.cuda.synchronize()

    K_steps, W = args.steps, max(args.warmup, 3)
    for i in range(W):
        step(i)
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)

    def timed_region(fn, n, first=0):
        """n calls of fn between two events on the launching stream, a barrier and a device synchronise on both sides."""
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        a.record()
        for i in range(n):
            fn(first + i)
        b.record()
        barrier()
        return a.elapsed_time(b)

    def repeated(fn, n, seconds, max_regions=2000):
        """The n-step region repeated until `seconds` of device time have been measured (every rank runs the same
        number of regions: the count comes from rank 0's first region).  Returns the per-region times."""
        first = timed_region(fn, n, W)
        cnt = R.max_over_ranks(me, [first], device=dev)[0]
        n_regions = int(min(max_regions, max(5, np.ceil(seconds * 1e3 / max(cnt, 1e-3)))))
        return [first] + [timed_region(fn, n, W + (r + 1) * n) for r in range(n_regions - 1)]

    # ---- timed region 1: device-resident inputs.  A region is exactly K steps from a drained stream to a drained
    # stream; it is repeated and the MEDIAN region is the reported value (a 20-step region lasts under a millisecond).
    t0 = time.time()
    regions = repeated(step, K_steps, args.seconds)
    # ---- the same region with plainly serialised launches
    regions_serial = repeated(lambda i: step(i, 0), K_steps, args.seconds / 4)
    # ---- one long region: the launch pipeline in steady state (labelled as such, never the headline)
    n_long = max(K_steps, args.steady_steps)
    ms_long = timed_region(step, n_long, W)

    # ---- the split-T kernel alone, per launch (events recorded inside the library call, serialised launches)
    n_iso = max(K_steps, 50)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_iso)]
    for a, b in evs:
        a.record(); b.record()
    barrier()
    for i in range(n_iso):
        S.stief_time_next_decode_kernel(*evs[i])
        step(W + i, 0)
    barrier()
    kern_ms = [a.elapsed_time(b) for a, b in evs]

    # ---- end to end through the host-buffer entry point
    staging = torch.empty(S.stief_host_staging_bytes(B, Hq, Hkv), dtype=torch.uint8, device=dev)
    qh = [q.cpu().pin_memory() for q in qs]
    kh = [(k.cpu().pin_memory(), v.cpu().pin_memory()) for k, v in kvs]
    out_h = torch.empty(B, Hq, 128, dtype=torch.bfloat16).pin_memory()

    def step_host(i):
        S.stief_decode_step_host(layers[i % n_caches], batch, qh[i % n_in], kh[i % n_in][0], kh[i % n_in][1], staging, ws,
                                 out_h, num_parts=ns, status=status, flags=0)
        torch.cuda.current_stream().synchronize()       # the caller reads out_h after every step

    for i in range(W):
        step_host(i)
    regions_host = repeated(step_host, K_steps, args.seconds / 4)
    t1 = time.time()
    if rank == 0:
        sampler.stop()
    assert int(status.item()) == 0, f"device status {int(status.item())}"

    # ---- context for the fraction: what a kernel that only reads gets from HBM (the peak in the denominator is a copy)
    read_gbs = None
    if rank == 0:
        scratch = torch.empty(2 << 30, dtype=torch.uint8, device=dev)      # one launch reads 2 GiB: launch cost is out of the picture
        for _ in range(2):
            S.stief_measure_read_stream(scratch, status)
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        r0.record()
        for _ in range(5):
            S.stief_measure_read_stream(scratch, status)
        r1.record()
        torch.cuda.synchronize()
        read_gbs = 5 * scratch.numel() / (r0.elapsed_time(r1) * 1e-3) / 1e9
        del scratch
        assert int(status.item()) == 0

    # ---- max over ranks, region by region; then the median region
    def med(v):
        v = R.max_over_ranks(me, v, device=dev)
        return float(np.median(v)), float(min(v)), float(max(v)), len(v)

    ms, ms_min, ms_max, n_reg = med(regions)
    ms_serial, _, _, n_reg_serial = med(regions_serial)
    ms_host, ms_host_min, ms_host_max, n_reg_host = med(regions_host)
    kern_isolated_ms, ms_long = R.max_over_ranks(me, [float(np.mean(kern_ms)), ms_long], device=dev)
    kern_avg_ms = ms / K_steps          # one launch per step: the timed region divided by its launches

    if rank == 0:
        hbm_peak, tf_peak, peak_kind = measured_peaks()
        sb = step_bytes(cfg)
        gbs = lambda region_ms, n=K_steps: world * sb * n / (region_ms * 1e-3) / 1e9
        value = gbs(ms)
        e2e = gbs(ms_host)
        achieved = sb / (kern_avg_ms * 1e-3) / 1e9
        # counters exist for the config-2 kernel at its own ranks only; any other workload reports null unless told
        traffic, traffic_source = args.traffic, (args.traffic_source if args.traffic is not None else None)
        if traffic is None and args.workload == "config2" and not args.ranks and args.num_parts in (None, 0):
            traffic, traffic_source = CAPTURED_TRAFFIC, CAPTURED_TRAFFIC_SOURCE
        pf_ms = float(np.median(prefill_ms))
        n_tok = sum(seq_lengths(cfg))
        pf_bytes = n_tok * Hkv * (2 * 128 * 2 + 2 * (r_k + r_v))
        pf_flops = 2.0 * n_tok * Hkv * 128 * (r_k + r_v)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K_steps, "warmup": W,
            "ms_per_step": ms / K_steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "dtype_note": "bf16 cache and tensor-core operands, fp32 accumulate", "data": "synthetic",
            "config": {"workload": cfg["name"] + ", 64-token pages, shuffled block tables; step = append + query projection + "
                                   "split-T attention + combine, one launch",
                       "global_batch": B * world, "seq_len": T, "r_k": r_k, "r_v": r_v, "num_parts": ns,
                       "launch": ("programmatic dependent launch: each step's kernel may start while the previous step's drains"
                                  if overlap else "serialised launches"),
                       "l2": f"steps rotate over {n_caches} layer caches of {sb / 2**20:.0f} MiB each (> 126 MB L2)",
                       "timing": f"value = median of {n_reg} timed regions of exactly {K_steps} steps, each from a drained stream "
                                 "to a drained stream (barrier + synchronise on both sides), max over ranks per region",
                       "parallelism": f"replicas x{world} (independent batches, no collective)"},
            "regions": {"count": n_reg, "median_ms": ms, "min_ms": ms_min, "max_ms": ms_max,
                        "value_at_min_ms": gbs(ms_min), "value_at_max_ms": gbs(ms_max)},
            "tokens_per_s": world * B * K_steps / (ms * 1e-3), "seq_lens": seq_lengths(cfg) if cfg.get("ragged") else None,
            "frac_of_hbm_peak": value / world / hbm_peak, "hbm_peak_gbs": hbm_peak, "peak_kind": peak_kind,
            "frac_of_hbm_spec_8000": value / world / 8000.0,
            "read_only_stream": {"gbs": read_gbs, "frac_of_it": value / world / read_gbs if read_gbs else None,
                                 "what": "the decode kernel's streaming skeleton without its arithmetic over a 2 GiB buffer "
                                         "(stief_measure_read_stream, CUDA events): what a read-only kernel gets from HBM, as context "
                                         "for a fraction whose denominator is a copy"},
            "e2e": {"value": e2e, "unit": UNIT, "h2d_bytes_per_step": (B * Hq + 2 * B * Hkv) * 128 * 2,
                    "d2h_bytes_per_step": B * Hq * 128 * 2, "ms_per_step": ms_host / K_steps,
                    "regions": {"count": n_reg_host, "median_ms": ms_host, "min_ms": ms_host_min, "max_ms": ms_host_max},
                    "transfer": "q, k_new, v_new and out are pinned mapped HOST buffers handed to stief_decode_step_host: the kernel "
                                "reads and writes them across the bus itself; the stream is synchronised after every step",
                    "tokens_per_s": world * B * K_steps / (ms_host * 1e-3)},
            "gpu_launches": K_steps,
            "roofline": {"bound": "hbm", "kernel": f"decode_persistent_kernel<{r_k},{r_v}>", "achieved": achieved, "peak": hbm_peak,
                         "unit": "GB/s", "frac": achieved / hbm_peak, "peak_kind": peak_kind, "traffic": traffic,
                         "traffic_source": traffic_source,
                         "bytes_per_launch": sb, "avg_launch_ms": kern_avg_ms,
                         "isolated_launch_ms": kern_isolated_ms, "isolated_min_launch_ms": float(min(kern_ms)),
                         "isolated_frac": sb / (kern_isolated_ms * 1e-3) / 1e9 / hbm_peak},
            "serial_launches": {"value": gbs(ms_serial), "unit": UNIT, "ms_per_step": ms_serial / K_steps, "regions": n_reg_serial,
                                "frac_of_hbm_peak": gbs(ms_serial) / world / hbm_peak},
            "steady_state": {"what": f"ONE region of {n_long} back-to-back overlapped steps: the launch pipeline in steady state, "
                                     "where the first launch's ramp and the last one's tail no longer count; not the headline",
                             "steps": n_long, "ms_per_step": ms_long / n_long, "value": gbs(ms_long, n_long), "unit": UNIT,
                             "frac_of_hbm_peak": gbs(ms_long, n_long) / world / hbm_peak},
            "prefill": {"ms_per_layer": pf_ms, "gbs": pf_bytes / (pf_ms * 1e-3) / 1e9, "frac_of_hbm_peak": pf_bytes / (pf_ms * 1e-3) / 1e9 / hbm_peak,
                        "tflops": pf_flops / (pf_ms * 1e-3) / 1e12, "frac_of_bf16_peak": pf_flops / (pf_ms * 1e-3) / 1e12 / tf_peak,
                        "workload": f"K,V [B={B},T={T},Hkv={Hkv},128] bf16 -> paged cache; per-layer time over back-to-back "
                                    f"overlapped launches on {n_caches} layers",
                        "kernel": "prefill_tc_kernel (TMA + tcgen05/TMEM)", "bound": "hbm"},
            "clocks": sampler.summary(t0, t1),
        }
        if not args.no_cpu_baseline:
            # world > 1: the other ranks wait in the final barrier meanwhile, so the sample is kept short
            line["cpu_baseline"] = cpu_baseline(cfg, seconds_budget=10.0 if world == 1 else 3.0)
        print(json.dumps(line))
    R.finish(me)


# ------------------------------------------------------------------------------------------------
# where a lone decode launch spends its time: per-CTA time stamps written by the kernel itself
# ------------------------------------------------------------------------------------------------
def run_trace(args):
    import paper_2601_21686_b200 as S
    from paper_2601_21686_b200 import inputs as I
    from paper_2601_21686_b200 import build as Bld

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    Bld.build()
    S.lib()
    cfg = dict(SINGLE_LAYER[args.workload])
    if args.ranks:
        cfg["r_k"], cfg["r_v"] = (int(x) for x in args.ranks.split(","))
    B, Hq, Hkv, T, r_k, r_v = (cfg[k] for k in ("B", "Hq", "Hkv", "T", "r_k", "r_v"))
    n_caches = args.caches
    layers, batch, status, _ = build_caches(cfg, n_caches, dev, S, I)
    ns = args.num_parts or S.stief_decode_num_parts()
    ws = torch.empty(S.stief_decode_workspace_bytes(B, Hq, Hkv, r_v, ns) // 4, dtype=torch.float32, device=dev)
    S.stief_decode_workspace_init(ws)
    out = torch.empty(B, Hq, 128, dtype=torch.bfloat16, device=dev)
    q = I.queries(SEED, 0, B, Hq, scale=1.0 / np.sqrt(128.0), device=dev)
    k_new, v_new = I.new_token_kv(SEED, 0, B, Hkv, device=dev)
    n = max(args.steps, 20)
    for i in range(5):
        S.stief_decode_step(layers[i % n_caches], batch, q, k_new, v_new, ws, out, num_parts=ns, status=status)
    torch.cuda.synchronize()
    names = ["entry", "partition known", "first page request", "first projections done", "first page landed", "last page request",
             "last page consumed", "last partial stored", "last combine done", "exit", "last arrival counted"]
    rel, dur_ev, spans, segs, combs = [], [], [], [], []
    for i in range(n):
        tr = torch.zeros(ns, S.TRACE_SLOTS, dtype=torch.int64, device=dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); e1.record()
        torch.cuda.synchronize()
        S.stief_trace_next_decode_kernel(tr)
        S.stief_time_next_decode_kernel(e0, e1)
        S.stief_decode_step(layers[i % n_caches], batch, q, k_new, v_new, ws, out, num_parts=ns, status=status)
        torch.cuda.synchronize()
        t = tr.cpu().numpy().astype(np.float64)
        stamps = np.concatenate([t[:, :10], t[:, 12:13]], axis=1)
        t0 = stamps[:, 0].min()
        r = np.where(stamps > 0, (stamps - t0) * 1e-3, np.nan)          # microseconds after the first CTA's entry
        rel.append(r)
        dur_ev.append(e0.elapsed_time(e1) * 1e3)
        spans.append(np.nanmax(r[:, 9]))
        segs.append(t[:, 10])
        combs.append(t[:, 11])
    assert int(status.item()) == 0
    chain = None
    if args.trace_chain:
        # a chain of overlapped launches with the time stamps of two consecutive kernels: when does the next kernel's CTA
        # enter an SM relative to the previous kernel's CTA leaving it, and how long is the SM without page traffic
        ov = S.STIEF_DECODE_OVERLAP_PREVIOUS
        gaps, idle, period = [], [], []
        phases = {k_: [] for k_ in ("last_page_to_partial", "partial_to_arrived", "arrived_to_exit", "entry_to_partition",
                                    "partition_to_first_request", "first_request_to_landed")}
        for rep_ in range(10):
            trs = [torch.zeros(ns, S.TRACE_SLOTS, dtype=torch.int64, device=dev) for _ in range(2)]
            torch.cuda.synchronize()
            for i in range(8):
                if i in (5, 6):
                    S.stief_trace_next_decode_kernel(trs[i - 5])
                S.stief_decode_step(layers[i % n_caches], batch, q, k_new, v_new, ws, out, num_parts=ns, status=status,
                                    flags=ov if i else 0)
            torch.cuda.synchronize()
            a_, b_ = (t_.cpu().numpy().astype(np.float64) for t_ in trs)
            a_, b_ = a_[a_[:, 0] > 0], b_[b_[:, 0] > 0]
            exit_by_sm = {int(r[13]): r[9] for r in a_}
            last_page_by_sm = {int(r[13]): r[6] for r in a_}
            for r in b_:
                sm = int(r[13])
                if sm in exit_by_sm:
                    gaps.append((r[0] - exit_by_sm[sm]) * 1e-3)          # previous CTA's exit -> this CTA's entry on the SM
                    idle.append((r[4] - last_page_by_sm[sm]) * 1e-3)     # previous CTA's last page consumed -> first page landed
            period.append((np.median(b_[:, 0]) - np.median(a_[:, 0])) * 1e-3)
            for x_ in (a_, b_):                                           # slots: see stief.h
                phases["last_page_to_partial"] += list((x_[:, 7] - x_[:, 6]) * 1e-3)
                phases["partial_to_arrived"] += list((x_[:, 12] - x_[:, 7]) * 1e-3)
                phases["arrived_to_exit"] += list((x_[:, 9] - x_[:, 12]) * 1e-3)
                phases["entry_to_partition"] += list((x_[:, 1] - x_[:, 0]) * 1e-3)
                phases["partition_to_first_request"] += list((x_[:, 2] - x_[:, 1]) * 1e-3)
                phases["first_request_to_landed"] += list((x_[:, 4] - x_[:, 2]) * 1e-3)
        chain = {"what": "overlapped chain, two consecutive kernels traced, matched by SM",
                 "exit_to_next_entry_us": {"median": float(np.median(gaps)), "p90": float(np.percentile(gaps, 90))},
                 "sm_without_page_traffic_us": {"median": float(np.median(idle)), "p90": float(np.percentile(idle, 90))},
                 "entry_to_entry_us": float(np.median(period)),
                 "phases_us_median_p90": {k_: [float(np.median(v_)), float(np.percentile(v_, 90))] for k_, v_ in phases.items()}}
    rel = np.stack(rel)                                                  # [launch, cta, slot]
    if args.trace_dump:                                                  # per-CTA table of the last launch, one line per CTA
        with open(args.trace_dump, "w") as f:
            f.write("cta segments combines " + " ".join(n.replace(" ", "_") for n in names) + "\n")
            for cta in range(ns):
                f.write(f"{cta} {int(segs[-1][cta])} {int(combs[-1][cta])} " + " ".join(f"{x:.3f}" for x in rel[-1, cta]) + "\n")
    hbm_peak, _, peak_kind = measured_peaks()
    sb = step_bytes(cfg)
    rows = {}
    for k, name in enumerate(names):
        x = rel[:, :, k]
        rows[name] = {"median_over_ctas_us": float(np.nanmedian(np.nanmedian(x, axis=1))),
                      "last_cta_us": float(np.nanmedian(np.nanmax(x, axis=1))),
                      "first_cta_us": float(np.nanmedian(np.nanmin(x, axis=1)))}
    print(json.dumps({
        "what": "time stamps written by decode_persistent_kernel itself (GPU nanosecond timer), microseconds after the first CTA's "
                "entry; one serialised launch at a time, median over launches; per point: median CTA, first CTA, last CTA",
        "workload": cfg["name"], "launches": n, "num_parts": ns, "points": rows,
        "kernel_span_us": float(np.median(spans)), "event_timed_launch_us": float(np.median(dur_ev)),
        "outside_the_kernel_us": float(np.median(dur_ev) - np.median(spans)),
        "roofline_time_us": sb / hbm_peak / 1e3, "peak_kind": peak_kind, "bytes_per_launch": sb,
        "stream_phase_us": {"median_cta": float(np.nanmedian(rel[:, :, 6] - rel[:, :, 4])),
                            "effective_gbs_over_first_landed_to_last_consumed":
                                sb / (float(np.nanmedian(np.nanmax(rel[:, :, 6], axis=1) - np.nanmin(rel[:, :, 4], axis=1))) * 1e-6) / 1e9},
        "chain": chain,
        "segments_per_cta": {"mean": float(np.mean(segs)), "max": float(np.max(segs))},
        "combines_per_cta": {"mean": float(np.mean(combs)), "max": float(np.max(combs))}}))


# ------------------------------------------------------------------------------------------------
# config 2 on the integer-quantised cache, 8-bit or 4-bit codes (a measurement case, not the headline line)
# ------------------------------------------------------------------------------------------------
def run_quant(args, bits):
    import paper_2601_21686_b200 as S
    from paper_2601_21686_b200 import inputs as I
    from paper_2601_21686_b200 import build as Bld

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    Bld.build()
    S.lib()
    hbm_peak, tf_peak, peak_kind = measured_peaks()
    cfg = dict(SINGLE_LAYER["config2"])
    if args.ranks:
        cfg["r_k"], cfg["r_v"] = (int(x) for x in args.ranks.split(","))
    B, Hq, Hkv, T, r_k, r_v = (cfg[k] for k in ("B", "Hq", "Hkv", "T", "r_k", "r_v"))
    n_caches = args.caches
    pg = I.make_paging(SEED, [T] * B, reserve_tokens=1)
    batch = S.Batch(torch.from_numpy(pg.block_table).to(dev), torch.from_numpy(pg.seq_lens).to(dev))
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    layers, inputs = [], []
    for l in range(n_caches):
        U_k, U_v = I.stiefel_bases(SEED, l, Hkv, r_k, r_v)
        K = I.lowrank_keys(SEED, l, B, T, Hkv, device=dev)
        V = I.gaussian_kv(SEED, I.TAG_V, l, B, T, Hkv, device=dev)
        # CALIBRATION INPUT, outside every timed region: the static key parameters the caller must bring (min / max of
        # the prompt's own projected keys per head and 64-channel group, widened by 25 %).  A real deployment takes
        # them from calibration data; this einsum only manufactures that input and is no part of the measured path.
        Kd = torch.einsum("bthd,hdr->bthr", K.float(), U_k.to(dev).float())
        groups = [(lo, min(lo + 64, r_k)) for lo in range(0, r_k, 64)]
        mn = torch.stack([Kd[..., lo:hi].amin(dim=(0, 1, 3)) for lo, hi in groups], -1)       # [Hkv, groups]
        mx = torch.stack([Kd[..., lo:hi].amax(dim=(0, 1, 3)) for lo, hi in groups], -1)
        kpar = torch.stack([(mx - mn) * 1.25 / float(2 ** bits - 1), mn * 1.25], -1).contiguous()
        del Kd
        layers.append(S.QLayer(Hq, Hkv, r_k, r_v, U_k.to(dev), U_v.to(dev), kpar,
                               torch.zeros(pg.num_pages, Hkv, 64, S.qkey_row_bytes(r_k, bits), dtype=torch.uint8, device=dev),
                               torch.zeros(pg.num_pages, Hkv, r_v, 64 if bits == 8 else 32, dtype=torch.uint8, device=dev),
                               torch.zeros(pg.num_pages, Hkv, 64, S.qgroups(r_v), 2, dtype=torch.float32, device=dev)))
        S.stief_q_prefill_compress(bits, layers[l], batch, K, V, status=status)
        inputs.append((K, V))
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 3
    e0.record()
    for r in range(reps):
        for l in range(n_caches):
            S.stief_q_prefill_compress(bits, layers[l], batch, inputs[l][0], inputs[l][1], status=status,
                                        flags=S.STIEF_PREFILL_OVERLAP_PREVIOUS if (r or l) else 0)
    e1.record()
    torch.cuda.synchronize()
    pf_ms = e0.elapsed_time(e1) / (reps * n_caches)
    del inputs
    ws = torch.empty(S.stief_decode_workspace_bytes(B, Hq, Hkv, r_v, 0) // 4, dtype=torch.float32, device=dev)
    S.stief_decode_workspace_init(ws)
    out = torch.empty(B, Hq, 128, dtype=torch.bfloat16, device=dev)
    n_in = 8
    qs = [I.queries(SEED, 0, B, Hq, scale=1.0 / np.sqrt(128.0), device=dev, step=i) for i in range(n_in)]
    kvs = [I.new_token_kv(SEED, 0, B, Hkv, device=dev, step=i) for i in range(n_in)]

    overlap = S.STIEF_DECODE_OVERLAP_PREVIOUS if (args.overlap and n_caches >= 2) else 0

    def step(i):
        S.stief_q_decode_step(bits, layers[i % n_caches], batch, qs[i % n_in], kvs[i % n_in][0], kvs[i % n_in][1], ws, out,
                               status=status, flags=overlap)

    K_steps, W = min(args.steps, 2000), max(args.warmup, 3)
    for i in range(W):
        step(i)
    torch.cuda.synchronize()
    e0.record()
    for i in range(K_steps):
        step(W + i)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    assert int(status.item()) == 0, f"device status {int(status.item())}"
    per_unit = S.qkey_row_bytes(r_k, bits) + r_v * bits // 8 + 8 * S.qgroups(r_v)
    sb = B * Hkv * (T + 1) * per_unit
    gbs = sb * K_steps / (ms * 1e-3) / 1e9
    pf_bytes = B * T * Hkv * (2 * 128 * 2 + per_unit)
    print(json.dumps({
        "metric": f"q{bits}_decode_attn_effective_hbm_gbs", "value": gbs, "unit": UNIT, "n_gpus": 1, "steps": K_steps, "warmup": W,
        "ms_per_step": ms / K_steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": f"u{bits}",
        "dtype_note": f"{bits}-bit codes as integer tensor-core operands (s8 x u8 -> s32), fp32 softmax and accumulation", "data": "synthetic",
        "config": {"workload": cfg["name"] + f" on the {bits}-bit quantised cache ({per_unit} bytes per token and KV head instead of {2 * (r_k + r_v)}); "
                               "step = append + query projection + split-T attention + combine, one launch"
                               + (", overlapped launches" if overlap else ""), "l2": f"steps rotate over {n_caches} layer caches"},
        "tokens_per_s": B * K_steps / (ms * 1e-3), "frac_of_hbm_peak": gbs / hbm_peak, "hbm_peak_gbs": hbm_peak, "peak_kind": peak_kind,
        "bytes_per_step": sb, "gpu_launches": K_steps,
        "same_step_in_bf16_cache_bytes_gbs": B * Hkv * (T + 1) * 2 * (r_k + r_v) * K_steps / (ms * 1e-3) / 1e9,
        "prefill": {"ms_per_layer": pf_ms, "gbs": pf_bytes / (pf_ms * 1e-3) / 1e9, "frac_of_hbm_peak": pf_bytes / (pf_ms * 1e-3) / 1e9 / hbm_peak}}))


# ------------------------------------------------------------------------------------------------
# a chunk of causal queries over the compressed cache (chunked prefill): a measurement case, not the headline line
# ------------------------------------------------------------------------------------------------
def run_mq(args):
    import paper_2601_21686_b200 as S
    from paper_2601_21686_b200 import inputs as I
    from paper_2601_21686_b200 import build as Bld

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    Bld.build()
    S.lib()
    hbm_peak, tf_peak, peak_kind = measured_peaks()
    cfg = dict(SINGLE_LAYER["config2"])
    if args.ranks:
        cfg["r_k"], cfg["r_v"] = (int(x) for x in args.ranks.split(","))
    B, Hq, Hkv, T, r_k, r_v = (cfg[k] for k in ("B", "Hq", "Hkv", "T", "r_k", "r_v"))
    n_q = args.n_q
    pg = I.make_paging(SEED, [T] * B, reserve_tokens=1)
    batch = S.Batch(torch.from_numpy(pg.block_table).to(dev), torch.from_numpy(pg.seq_lens).to(dev))
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    n_caches = max(1, min(args.caches, 2))
    layers = []
    for l in range(n_caches):
        U_k, U_v = I.stiefel_bases(SEED, l, Hkv, r_k, r_v)
        layer = S.Layer(Hq, Hkv, r_k, r_v, U_k.to(dev), U_v.to(dev),
                        torch.zeros(pg.num_pages, Hkv, 64, r_k, dtype=torch.bfloat16, device=dev),
                        torch.zeros(pg.num_pages, Hkv, 64, r_v, dtype=torch.bfloat16, device=dev))
        K = I.lowrank_keys(SEED, l, B, T, Hkv, device=dev)
        V = I.gaussian_kv(SEED, I.TAG_V, l, B, T, Hkv, device=dev)
        S.stief_prefill_compress(layer, batch, K, V, status=status)
        del K, V
        layers.append(layer)
    qs = [I.normal_bf16(I.stream_key(SEED, I.TAG_Q, 100 + i), (B, n_q, Hq, 128), device=dev) for i in range(2)]
    out = torch.empty(B, n_q, Hq, 128, dtype=torch.bfloat16, device=dev)
    n_split = S.stief_mq_num_splits(B, n_q, Hq, Hkv, batch.block_table.shape[1]) if args.splits is None else args.splits
    ws = torch.empty(max(S.stief_mq_workspace_bytes(B, n_q, Hq, r_v, n_split) // 4, 1), dtype=torch.float32, device=dev) if n_split > 1 else None
    torch.cuda.synchronize()

    def step(i):
        S.stief_mq_attention(layers[i % n_caches], batch, qs[i % 2], out, status=status, workspace=ws, num_splits=n_split)

    K_steps, W = min(args.steps, 50 if n_q >= 256 else 2000), max(min(args.warmup, 5), 3)
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.3)
    for i in range(W):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record()
    for i in range(K_steps):
        step(W + i)
    e1.record()
    torch.cuda.synchronize()
    t1 = time.time()
    ms = e0.elapsed_time(e1) / K_steps
    sampler.stop()
    assert int(status.item()) == 0, f"device status {int(status.item())}"
    visible = sum(T - n_q + i + 1 for i in range(n_q))                     # cached positions each query row attends, summed
    flops = B * Hq * (2 * visible * (r_k + r_v) + n_q * 2 * 128 * (r_k + r_v))
    tflops = flops / (ms * 1e-3) / 1e12
    cache_bytes = B * Hkv * T * 2 * (r_k + r_v)
    print(json.dumps({
        "metric": "mq_attention_tflops", "value": tflops, "unit": "TFLOP/s", "n_gpus": 1, "steps": K_steps, "warmup": W,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "dtype_note": "bf16 tensor-core operands (tcgen05), fp32 accumulate in TMEM", "data": "synthetic",
        "config": {"workload": f"chunk of {n_q} causal query tokens per sequence at the end of a {T}-token compressed cache, "
                               f"B={B} Hq={Hq} Hkv={Hkv} r_k={r_k} r_v={r_v}: query projection + causal attention + back-projection"
                               + (f", page ranges split {n_split} ways + merge kernel" if n_split > 1 else ", one launch"),
                   "l2": f"steps alternate over {n_caches} layer caches of {cache_bytes / 2**20:.0f} MiB"},
        "query_tokens_per_s": B * n_q / (ms * 1e-3), "gpu_launches": K_steps * (2 if n_split > 1 else 1),
        "cache_read_gbs": cache_bytes / (ms * 1e-3) / 1e9, "cache_read_frac_of_hbm_peak": cache_bytes / (ms * 1e-3) / 1e9 / hbm_peak,
        "roofline": {"bound": "tensor", "kernel": "mq_attention_kernel", "achieved": tflops, "peak": tf_peak, "unit": "TFLOP/s",
                     "frac": tflops / tf_peak, "peak_kind": peak_kind, "traffic": None, "flops_per_launch": flops,
                     "avg_launch_ms": ms},
        "clocks": sampler.summary(t0, t1)}))


# ------------------------------------------------------------------------------------------------
# the 32-layer workloads: config 3 (decode steps over per-layer ranks) and config 5 (prefill + first decode)
# ------------------------------------------------------------------------------------------------
def run_multilayer(args):
    import paper_2601_21686_b200 as S
    from paper_2601_21686_b200 import inputs as I
    from paper_2601_21686_b200 import build as Bld

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    if int(os.environ.get("WORLD_SIZE", "1")) != 1:
        raise SystemExit("the multi-layer workloads run on one GPU")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    Bld.build()
    S.lib()
    hbm_peak, tf_peak, peak_kind = measured_peaks()
    Hq, Hkv, T, L = 32, 8, 32768, args.layers
    B = 4 if args.workload == "config3" else 2
    n_steps = args.steps if args.workload == "config3" else 1
    if args.rho is not None:
        # ranks from the library's own selector (Algorithm 2) on synthetic error surfaces of the shape the paper reports
        prof, _ = S.stief_select_ranks(L, I.RANK_SET, I.RANK_SET, args.rho, surfaces=I.error_surfaces(SEED, L))
    elif args.ranks:
        # every layer at the same ranks (not the named workload): separates what the mix of kernel variants costs
        pairs = [tuple(int(x) for x in pr.split(",")) for pr in args.ranks.split(";")]
        prof = [pairs[l % len(pairs)] for l in range(L)]
    else:
        prof = I.rank_profile(SEED)[:L]
    pg = I.make_paging(SEED, [T] * B, reserve_tokens=max(n_steps, 1) + 1)
    bt = torch.from_numpy(pg.block_table).to(dev)
    lens = torch.from_numpy(pg.seq_lens).to(dev)
    batch = S.Batch(bt, lens)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    layers, inputs = [], []
    for l, (r_k, r_v) in enumerate(prof):
        U_k, U_v = I.stiefel_bases(SEED, l, Hkv, r_k, r_v)
        layers.append(S.Layer(Hq, Hkv, r_k, r_v, U_k.to(dev), U_v.to(dev),
                              torch.zeros(pg.num_pages, Hkv, 64, r_k, dtype=torch.bfloat16, device=dev),
                              torch.zeros(pg.num_pages, Hkv, 64, r_v, dtype=torch.bfloat16, device=dev)))
        K = I.lowrank_keys(SEED, l, B, T, Hkv, device=dev)
        V = I.gaussian_kv(SEED, I.TAG_V, l, B, T, Hkv, device=dev)
        if args.workload == "config5":
            inputs.append((K, V))                 # all 32 layers' prompts stay resident (8.6 GB) for the timed prefill
        else:
            S.stief_prefill_compress(layers[l], batch, K, V, status=status)
            del K, V
    torch.cuda.synchronize()
    ws = torch.empty(S.stief_decode_workspace_bytes(B, Hq, Hkv, 128, 0) // 4, dtype=torch.float32, device=dev)
    S.stief_decode_workspace_init(ws)
    outs = [torch.empty(B, Hq, 128, dtype=torch.bfloat16, device=dev) for _ in range(L)]   # overlapped kernels never share an output
    n_in = 4
    qs = [[I.queries(SEED, l, B, Hq, scale=1.0 / np.sqrt(128.0), device=dev, step=i) for l in range(L)] for i in range(n_in)]
    kvs = [[I.new_token_kv(SEED, l, B, Hkv, device=dev, step=i) for l in range(L)] for i in range(n_in)]
    ov = S.STIEF_DECODE_OVERLAP_PREVIOUS

    def decode_step(i):
        """One token for every sequence: append + attention in every layer, then advance the lengths."""
        for l in range(L):
            k_new, v_new = kvs[i % n_in][l]
            S.stief_decode_step(layers[l], batch, qs[i % n_in][l], k_new, v_new, ws, outs[l], status=status, flags=ov if l else 0)
        S.stief_advance_seq_lens(lens, 1)

    cache_bytes_per_token = sum(Hkv * 2 * (rk + rv) for rk, rv in prof)      # per cached token, all layers
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.3)
    t0 = time.time()
    line = {"n_gpus": 1, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "data": "synthetic",
            "dtype": "bf16", "dtype_note": "bf16 cache and tensor-core operands, fp32 accumulate", "rank_profile": prof, "peak_kind": peak_kind, "hbm_peak_gbs": hbm_peak}
    if args.workload == "config3":
        W = 3
        for i in range(W):
            decode_step(i)
        lens.copy_(torch.from_numpy(pg.seq_lens).to(dev))          # the timed steps start from T again
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(n_steps):
            decode_step(W + i)
        e1.record()
        torch.cuda.synchronize()
        ms_eager = e0.elapsed_time(e1)
        # the same step replayed from a CUDA graph (the lengths advance on the device, so one captured step serves
        # every position): removes the host's per-launch cost, which the small-rank layers cannot hide
        lens.copy_(torch.from_numpy(pg.seq_lens).to(dev))
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        cap_stream = torch.cuda.Stream()
        cap_stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(cap_stream):
            with torch.cuda.graph(graph, stream=cap_stream):
                decode_step(0)
        torch.cuda.synchronize()
        for i in range(W):
            graph.replay()
        lens.copy_(torch.from_numpy(pg.seq_lens).to(dev))
        torch.cuda.synchronize()
        e0.record()
        for i in range(n_steps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        byt = sum(B * (T + s + 1) * cache_bytes_per_token for s in range(n_steps))
        gbs = byt / (ms * 1e-3) / 1e9
        line.update({"eager_launches": {"ms_per_step": ms_eager / n_steps, "value": byt / (ms_eager * 1e-3) / 1e9, "unit": UNIT,
                                        "tokens_per_s": B * n_steps / (ms_eager * 1e-3)},
                     "launch": "one captured CUDA graph per step (32 decode launches + the length update), replayed"})
        line.update({"metric": METRIC, "value": gbs, "unit": UNIT, "steps": n_steps, "warmup": W, "ms_per_step": ms / n_steps,
                     "tokens_per_s": B * n_steps / (ms * 1e-3), "frac_of_hbm_peak": gbs / hbm_peak,
                     "gpu_launches": n_steps * (L + 1), "bytes_per_step_first": B * (T + 1) * cache_bytes_per_token,
                     "config": {"workload": f"config3: {L}-layer decode step, per-layer ranks from the seeded profile, B={B} Hq={Hq} "
                                            f"Hkv={Hkv} d=128 T={T} growing by one token per step; step = for every layer append + "
                                            "attention (one launch each, overlapped within a step), then advance the lengths",
                                "global_batch": B, "seq_len": T, "l2": "a step streams 9.9 GB of cache: nothing survives in L2"}})
    else:
        pf = S.STIEF_PREFILL_OVERLAP_PREVIOUS
        for l in range(min(4, L)):                # warm-up on a few layers (they are rewritten below)
            S.stief_prefill_compress(layers[l], batch, inputs[l][0], inputs[l][1], status=status)
        decode_step(0)                            # loads every decode kernel variant; its rows are rewritten below
        lens.copy_(torch.from_numpy(pg.seq_lens).to(dev))
        torch.cuda.synchronize()
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record()
        for l in range(L):
            S.stief_prefill_compress(layers[l], batch, inputs[l][0], inputs[l][1], status=status, flags=pf if l else 0)
        e1.record()
        decode_step(0)
        e2.record()
        torch.cuda.synchronize()
        ms_pf, ms_dec = e0.elapsed_time(e1), e1.elapsed_time(e2)
        byt = sum(B * T * Hkv * (512 + 2 * (rk + rv)) for rk, rv in prof)
        flops = sum(2.0 * B * T * Hkv * 128 * (rk + rv) for rk, rv in prof)
        gbs = byt / (ms_pf * 1e-3) / 1e9
        line.update({"metric": "prefill_compress_effective_hbm_gbs", "value": gbs, "unit": UNIT, "steps": 1, "warmup": 1,
                     "ms_per_step": ms_pf, "ms_per_layer": ms_pf / L, "frac_of_hbm_peak": gbs / hbm_peak,
                     "tflops": flops / (ms_pf * 1e-3) / 1e12, "frac_of_bf16_peak": flops / (ms_pf * 1e-3) / 1e12 / tf_peak,
                     "prompt_tokens_per_s": B * T / (ms_pf * 1e-3), "gpu_launches": L,
                     "first_decode_step": {"ms": ms_dec, "gbs": B * (T + 1) * cache_bytes_per_token / (ms_dec * 1e-3) / 1e9},
                     "config": {"workload": f"config5: prefill compression of a {L}-layer prompt, K,V [B={B},T={T},Hkv={Hkv},128] bf16 per "
                                            "layer -> paged cache with per-layer ranks (one overlapped launch per layer), then the first decode step",
                                "global_batch": B, "seq_len": T, "l2": "every layer has its own 268 MB of inputs"}})
    torch.cuda.synchronize()
    sampler.stop()
    line["clocks"] = sampler.summary(t0, time.time())
    assert int(status.item()) == 0, f"device status {int(status.item())}"
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# the oracle, timed on the host cores (a reported baseline, and the `--impl reference` arm)
# ------------------------------------------------------------------------------------------------
def _oracle_sample(cfg, n_seq):
    """Inputs and oracle cache for the first n_seq sequences of the workload (CPU, fp64)."""
    from oracle import stief_oracle as O
    from paper_2601_21686_b200 import inputs as I
    Hq, Hkv, T, r_k, r_v = (cfg[k] for k in ("Hq", "Hkv", "T", "r_k", "r_v"))
    K = I.lowrank_keys(SEED, 0, n_seq, T, Hkv).double().numpy()
    V = I.gaussian_kv(SEED, I.TAG_V, 0, n_seq, T, Hkv).double().numpy()
    U_k, U_v = I.stiefel_bases(SEED, 0, Hkv, r_k, r_v)
    U_k, U_v = U_k.double().numpy(), U_v.double().numpy()
    Kd, Vd = O.compress_layer(K, V, U_k, U_v, [T] * n_seq)
    return O, I, Kd, Vd, U_k, U_v


def _oracle_step(O, I, cfg, n_seq, Kd, Vd, U_k, U_v, i):
    """One decode step of the oracle on the sample: append the new token's projected rows, then attend."""
    Hq, Hkv = cfg["Hq"], cfg["Hkv"]
    q = I.queries(SEED, 0, n_seq, Hq, scale=1.0 / np.sqrt(128.0), step=i).double().numpy()
    k_new, v_new = I.new_token_kv(SEED, 0, n_seq, Hkv, step=i)
    k_new, v_new = k_new.double().numpy(), v_new.double().numpy()
    t0 = time.perf_counter()
    Kd2, Vd2 = [], []
    for b in range(n_seq):
        kr = np.stack([O.compress(k_new[b, h][None], O.basis_of(U_k, h))[0] for h in range(Hkv)])[None]
        vr = np.stack([O.compress(v_new[b, h][None], O.basis_of(U_v, h))[0] for h in range(Hkv)])[None]
        Kd2.append(np.concatenate([Kd[b], kr], 0))
        Vd2.append(np.concatenate([Vd[b], vr], 0))
    out, _ = O.decode_layer(q, Kd2, Vd2, U_k, U_v, "b")
    return time.perf_counter() - t0, out


def _threads_used() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return int(max(n)) if n else 1
    except Exception:
        return 1


def cpu_baseline(cfg, seconds_budget=10.0):
    n_seq = 1
    O, I, Kd, Vd, U_k, U_v = _oracle_sample(cfg, n_seq)
    sb = n_seq * (cfg["T"] + 1) * cfg["Hkv"] * 2 * (cfg["r_k"] + cfg["r_v"])
    dts = []
    t_start = time.perf_counter()
    i = 0
    while i < 3 or (time.perf_counter() - t_start < seconds_budget and i < 150):
        dt, _ = _oracle_step(O, I, cfg, n_seq, Kd, Vd, U_k, U_v, i)
        dts.append(dt)
        i += 1
    best = min(dts)
    return {"value": sb / best / 1e9, "unit": UNIT, "cores": _threads_used(), "host_cores": os.cpu_count(), "kind": "oracle",
            "sample": f"{n_seq} of {cfg['B']} sequences of the same workload (all {cfg['Hq']} query heads, T={cfg['T']}), "
                      f"{len(dts)} decode steps (append + attention, fp64 numpy), best step",
            "s_per_step_sample": best, "tokens_per_s": n_seq / best}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = dict(CFG2)
    n_seq = 1
    O, I, Kd, Vd, U_k, U_v = _oracle_sample(cfg, n_seq)
    sb = n_seq * (cfg["T"] + 1) * cfg["Hkv"] * 2 * (cfg["r_k"] + cfg["r_v"])
    W, K_steps = max(args.warmup, 1), args.steps
    for i in range(W):
        _oracle_step(O, I, cfg, n_seq, Kd, Vd, U_k, U_v, i)
    total = 0.0
    for i in range(K_steps):
        dt, _ = _oracle_step(O, I, cfg, n_seq, Kd, Vd, U_k, U_v, W + i)
        total += dt
    value = sb * K_steps / total / 1e9
    sample = (f"each step = one decode step (append + attention, fp64 numpy) on {n_seq} of {cfg['B']} sequences of the workload "
              f"(all {cfg['Hq']} query heads, T={cfg['T']})")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
            "steps": K_steps, "warmup": W, "ms_per_step": total / K_steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "config2: Llama3-8B-shaped single-layer decode, B=4 Hq=32 Hkv=8 d=128 T=32768 r_k=r_v=64 (bounded sample)",
                       "sample": sample},
            "tokens_per_s": n_seq * K_steps / total,
            "cpu_baseline": {"value": value, "unit": UNIT, "kind": "oracle", "cores": _threads_used(), "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps per region (default 20; 128 for config3)")
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config2", choices=["config2", "config3", "config4a", "config4b", "config5"],
                    help="config2 is the headline line; the others are the remaining benchmark configurations")
    ap.add_argument("--num-parts", type=int, default=0, help="CTAs of the persistent decode kernel (0 = one per SM)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--q8", action="store_true", help="config 2 on the 8-bit quantised cache (measurement case)")
    ap.add_argument("--q4", action="store_true", help="config 2 on the 4-bit quantised cache (measurement case)")
    ap.add_argument("--ranks", default=None, help="r_k,r_v override for the single-layer workloads, e.g. 48,96; with config3/config5: every layer at these ranks, or several pairs separated by ; taken in turn")
    ap.add_argument("--layers", type=int, default=32, help="layers of the multi-layer workloads (config3, config5)")
    ap.add_argument("--no-overlap", dest="overlap", action="store_false",
                    help="launch every step's kernel fully serialised (no programmatic dependent launch)")
    ap.add_argument("--caches", type=int, default=N_CACHES, help="independent layer caches the steps rotate over")
    ap.add_argument("--mq", action="store_true", help="measure the multi-query (chunked prefill) attention kernel on the config-2 shape")
    ap.add_argument("--n-q", dest="n_q", type=int, default=2048, help="query tokens per sequence for --mq")
    ap.add_argument("--splits", type=int, default=None, help="--mq: parts per page range (default: the library's proposal)")
    ap.add_argument("--rho", type=float, default=None, help="multi-layer workloads: take the per-layer ranks from stief_select_ranks at this cache ratio instead of the seeded random profile")
    ap.add_argument("--traffic", type=float, default=None,
                    help="dram bytes (read + write) per launch of the split-T kernel from an ncu capture of the CURRENT kernel; "
                         "without it roofline.traffic is null")
    ap.add_argument("--traffic-source", default=None, help="where --traffic comes from (profile file and commit of the capture)")
    ap.add_argument("--trace", action="store_true",
                    help="single-layer workloads: per-CTA time stamps of lone decode launches (where the time of a launch goes)")
    ap.add_argument("--trace-chain", action="store_true", help="--trace: also trace two consecutive kernels of an overlapped chain")
    ap.add_argument("--trace-dump", default=None, help="--trace: also write the last launch's per-CTA table to this file")
    ap.add_argument("--seconds", type=float, default=0.6,
                    help="device time to collect by repeating the K-step timed region (the median region is reported)")
    ap.add_argument("--steady-steps", type=int, default=4000, help="steps of the one long region reported under steady_state")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 128 if args.workload == "config3" else (20 if not (args.q8 or args.q4 or args.mq) else 2000)
    if args.impl == "reference":
        run_reference(args)
    elif args.trace:
        run_trace(args)
    elif args.q8 or args.q4:
        run_quant(args, 8 if args.q8 else 4)
    elif args.mq:
        run_mq(args)
    elif args.workload in SINGLE_LAYER:
        run_ours(args)
    else:
        run_multilayer(args)


if __name__ == "__main__":
    main()
