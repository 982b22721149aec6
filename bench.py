#!/usr/bin/env python
"""Benchmark of the QAQ hot path (arXiv 2403.04643) on B200.

One step = one pass of the whole hot path over one synthetic LLaMA-7B-shaped KV cache
(default workload C3: 32 layers x batch 8 x 32 heads x 4096 tokens x head_dim 128):
per layer  outlier thresholds -> fused bit selection + outlier split + quantize + pack
(`qaq_quantize_append`) -> decode attention over the packed cache (`qaq_decode_attention`).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload C3]

Prints ONE JSON line (rank 0).  `value` = algorithmic GB/s of the whole step, summed over
ranks (each rank holds its own batch: weak scaling, no data-path collective).
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2403_04643_b200 import synth  # noqa: E402

# ncu counters of the main kernels (DRAM bytes and warp instructions per launch on the C3 layer shape) are read from
# profiles/counters_C3.json, which `bench.py --write-counters <ncu csv>` writes together with a hash of the kernel
# sources; they are reported only while that hash matches the sources, otherwise as null with the reason.
import hashlib

COUNTERS_JSON = os.path.join(ROOT, "profiles", "counters_C3.json")
CSRC = os.path.join(ROOT, "paper_2403_04643_b200", "csrc")
ISSUE_SLOTS_PER_CLOCK = 148 * 4
KERNEL_KEYS = {"quant_keys": "quant_kernel<128, 0, 0>", "quant_values": "quant_kernel<128, 0, 1>", "decode": "decode_kernel<128, 0>",
               "thr_scan": "thr_scan_kernel"}


def csrc_hash():
    h = hashlib.sha256()
    for f in sorted(os.listdir(CSRC)):
        if f.endswith((".cu", ".cuh")):
            with open(os.path.join(CSRC, f), "rb") as fh:
                h.update(f.encode()); h.update(fh.read())
    return h.hexdigest()[:16]


def load_counters():
    try:
        with open(COUNTERS_JSON) as f:
            c = json.load(f)
    except (OSError, ValueError):
        return None, "profiles/counters_C3.json not found"
    if c.get("csrc_hash") != csrc_hash():
        return None, "kernel sources changed since the counters were taken"
    return c, None


def write_counters(csv_path):
    """Parses an `ncu --csv` log with dram__bytes_read.sum, dram__bytes_write.sum, smsp__inst_executed.sum and
    gpu__time_duration.sum per launch and writes the per-kernel averages to profiles/counters_C3.json."""
    import csv
    rows = [r for r in csv.reader(open(csv_path)) if len(r) > 10]
    hdr = rows[0]
    ki, mi, vi, ii = hdr.index("Kernel Name"), hdr.index("Metric Name"), hdr.index("Metric Value"), hdr.index("ID")
    per = {}
    for r in rows[1:]:
        per.setdefault((r[ii], r[ki]), {})[r[mi]] = float(r[vi].replace(",", ""))
    out = {"csrc_hash": csrc_hash(), "source": os.path.basename(csv_path), "shape": "C3 layer: 256 (b,h) x 4096 tokens x 128", "kernels": {}}
    for key, pat in KERNEL_KEYS.items():
        ms = [m for (_, name), m in per.items() if pat in name]
        if not ms:
            continue
        avg = lambda k: sum(m.get(k, 0.0) for m in ms) / len(ms)
        out["kernels"][key] = {"launches": len(ms), "dram_bytes": avg("dram__bytes_read.sum") + avg("dram__bytes_write.sum"),
                               "warp_instr": avg("smsp__inst_executed.sum"), "time_us": avg("gpu__time_duration.sum") / 1e3}
    with open(COUNTERS_JSON, "w") as f:
        json.dump(out, f, indent=1)
        f.write("\n")
    print(json.dumps(out))


def issue_roofline(n, seconds, sm_mhz):
    if not n or not seconds or not sm_mhz:
        return None
    peak = ISSUE_SLOTS_PER_CLOCK * sm_mhz * 1e6
    return {"bound": "alu", "warp_instr_per_launch": n, "achieved": round(n / seconds / 1e9, 1), "peak": round(peak / 1e9, 1),
            "unit": "G warp-instr/s", "frac": round(n / seconds / peak, 3)}


METRIC = "QAQ quantize GB/s + packed decode-attn tokens/s, % of B200 HBM peak"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            with open(self.path) as f:
                for line in f:
                    parts = [p.strip() for p in line.split(",")]
                    if len(parts) < 6:
                        continue
                    try:
                        sm.append(float(parts[0])); mx.append(float(parts[1]))
                    except ValueError:
                        continue
                    for n, v in zip(names, parts[2:6]):
                        if v.lower().startswith("active"):
                            reasons.add(n)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out = {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}
        return out


# ----------------------------------------------------------------------------- byte accounting
def algorithmic_bytes(wl, st, n_layers_stats=1):
    """Per-layer algorithmic bytes of each stage from the cache statistics of one layer."""
    BH, T, D, W = wl.bh, wl.tokens, wl.head_dim, wl.window
    th = BH * T                                        # token-heads
    ntile = BH * math.ceil(T / 64)
    codes = st.code_bytes[0] + st.code_bytes[1]
    outl = 4 * (st.outliers[0] + st.outliers[1])
    meta = 2 * 5 * th + 2 * 16 * ntile                 # width + min/max per token and tensor; tile tables
    fp16 = 2 * 2 * D * th
    return {
        "thresholds": fp16,                            # one read of K and V
        "quantize": fp16 + (4 * W + 1) * th + codes + meta + outl,
        "decode": codes + meta + outl + BH * D * (2 + 4),
        "fp16": fp16,
    }


# ----------------------------------------------------------------------------- CPU baseline (oracle)
def oracle_sample(wl, hyper, n_bh, threads, device):
    """Times the oracle (thresholds + select + quantize + decode) on n_bh (b,h) of layer 0."""
    import numpy as np
    import oracle
    small = synth.scaled(wl, batch=1, heads=n_bh, layers=1)
    K, V = synth.make_kv(small, 0, device=device)
    q = synth.make_query(small, 0, device=device)
    ring, nv = synth.make_score_ring(small, 0, device=device)
    u16 = lambda t: t.cpu().contiguous().numpy().view(np.uint16)
    T, D = wl.tokens, wl.head_dim
    cK, cV = oracle.policy(hyper[0], hyper[1], hyper[2], T)
    args = (u16(K).reshape(n_bh, T, D), u16(V).reshape(n_bh, T, D), u16(q).reshape(n_bh, D),
            ring.cpu().numpy().reshape(n_bh, wl.window, T), nv.cpu().numpy().reshape(n_bh, T))
    kw = dict(alpha=wl.alpha, cK=cK, cV=cV, bmin=wl.bits_min, bmax=wl.bits_max, scale=1.0 / math.sqrt(D),
              n_threads=threads, out_cap=max(1024, T * D // 2), want_scores=False, materialize=False)

    def run():
        t0 = time.perf_counter()
        r = oracle.run_batch(*args, **kw)
        return time.perf_counter() - t0, r
    return run


def per_th_bytes(wl, mean_bits=(4.0, 3.0)):
    """Algorithmic bytes per token-head of the whole step at nominal widths (for the oracle's GB/s)."""
    D, W = wl.head_dim, wl.window
    codes = D * (mean_bits[0] + mean_bits[1]) / 8
    outl = 2 * wl.alpha * D * 4
    fp16 = 4 * D
    return fp16 + (fp16 + 4 * W + 1 + codes + 10 + outl) + (codes + 10 + outl)


def config_of(wl, hyper):
    """What both arms of the benchmark report as their configuration."""
    return {"workload": wl.name, "layers": wl.layers, "batch": wl.batch, "heads": wl.heads, "head_dim": wl.head_dim,
            "tokens": wl.tokens, "window": wl.window, "alpha": wl.alpha, "widths": [wl.bits_min, wl.bits_max],
            "sigmaS_max": hyper[0], "sigmaX_max": hyper[1], "qnorm2": hyper[2]}


# ----------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C3", choices=sorted(synth.CONFIGS))
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (0 = the workload's)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true")
    ap.add_argument("--extras", default="", help="run only the extra points whose name starts with this")
    ap.add_argument("--streams", type=int, default=3, help="streams the independent layers of a step are spread over")
    ap.add_argument("--no-graph", action="store_true", help="launch the timed steps on the stream instead of replaying a CUDA graph")
    ap.add_argument("--write-counters", default="", help="parse an ncu --csv log and write profiles/counters_C3.json (no GPU needed)")
    args = ap.parse_args()
    if args.write_counters:
        write_counters(args.write_counters)
        return 0
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    wl = synth.CONFIGS[args.workload]
    if args.layers > 0:
        wl = synth.scaled(wl, layers=args.layers)
    peak, peak_kind = measured_peaks()
    from paper_2403_04643_b200.calibrate import frozen
    hyper = frozen(args.workload)       # (sigmaS_max, sigmaX_max, qnorm2) frozen per workload in hyper.json

    if args.impl == "reference":
        if rank != 0:
            return 0
        return reference_arm(args, wl, hyper)

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    from paper_2403_04643_b200 import qaq
    from paper_2403_04643_b200.calibrate import calibrate, qnorm2_of_queries
    from paper_2403_04643_b200 import dist as qdist
    qaq.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    BH, T, D, W, L = wl.bh, wl.tokens, wl.head_dim, wl.window, wl.layers
    scale = 1.0 / math.sqrt(D)
    cfg = qaq.make_config(wl.batch, wl.heads, D, T, wl.bits_min, wl.bits_max, W, wl.alpha)
    # ---- resident inputs (each rank its own batch: seed offset by rank)
    wl_r = synth.scaled(wl, seed=qdist.rank_seed(wl.seed, rank))
    layers = []
    for l in range(L):
        K, V = synth.make_kv(wl_r, l, device=dev)
        q = synth.make_query(wl_r, l, device=dev)
        ring, nv = synth.make_score_ring(wl_r, l, device=dev)
        layers.append(dict(K=K, V=V, q=q, ring=ring, nv=nv, cache=qaq.Cache(cfg),
                           thr=torch.empty((BH, 4), dtype=torch.float32, device=dev),
                           out=torch.empty((BH, D), dtype=torch.float32, device=dev)))
    torch.cuda.synchronize()
    # ---- hyper-parameters: calibrated once on layer 0 (mean widths ~4 / ~3)
    L0 = layers[0]
    qaq.qaq_outlier_thresholds(cfg, L0["K"], L0["V"], L0["thr"])
    # Section 4.1: the upper 10 % quantile of the squared (scaled) query norms, taken on the device over this run's queries
    qn_measured = qnorm2_of_queries(wl_r, dev, layers=L)
    if hyper is not None:
        sS, sX, hyper_qn = hyper
        pol = qaq.qaq_policy_from_hyper(sS, sX, hyper_qn, T)
        hyper_source = "paper_2403_04643_b200/hyper.json"
    else:               # a workload without frozen values: bisection to mean widths (4, 3) on layer 0
        hyper_qn = qn_measured
        sS, sX, pol = calibrate(cfg, L0["K"], L0["V"], L0["ring"], L0["nv"], L0["thr"], T, hyper_qn)
        hyper_source = "calibrated in this run"

    # layers are independent problems: outside the per-stage timing pass they are spread over a few streams, so that
    # the short, latency-bound kernels of one layer (threshold sample / select, merge) overlap another layer's long ones
    side = [torch.cuda.Stream(device=dev) for _ in range(max(0, args.streams - 1))]

    def step(timers=None):
        if timers is None and side:
            main = torch.cuda.current_stream()
            lanes = [main] + side
            for sd in side:
                sd.wait_stream(main)
            for i, Ly in enumerate(layers):
                with torch.cuda.stream(lanes[i % len(lanes)]):
                    c = Ly["cache"]
                    c.reset()
                    qaq.qaq_outlier_thresholds(cfg, Ly["K"], Ly["V"], Ly["thr"])
                    qaq.qaq_quantize_append(c, Ly["K"], Ly["V"], Ly["thr"], policy=pol, ring=Ly["ring"], nvalid=Ly["nv"])
                    qaq.qaq_decode_attention(c, Ly["q"], scale, out=Ly["out"])
            for sd in side:
                main.wait_stream(sd)
            return
        for Ly in layers:
            c = Ly["cache"]
            c.reset()
            if timers: timers["thr"][0].append(ev())
            qaq.qaq_outlier_thresholds(cfg, Ly["K"], Ly["V"], Ly["thr"])
            if timers: timers["thr"][1].append(ev()); timers["quant"][0].append(timers["thr"][1][-1])
            qaq.qaq_quantize_append(c, Ly["K"], Ly["V"], Ly["thr"], policy=pol, ring=Ly["ring"], nvalid=Ly["nv"])
            if timers: timers["quant"][1].append(ev()); timers["dec"][0].append(timers["quant"][1][-1])
            qaq.qaq_decode_attention(c, Ly["q"], scale, out=Ly["out"])
            if timers: timers["dec"][1].append(ev())

    def ev():
        e = torch.cuda.Event(enable_timing=True)
        e.record()
        return e

    def barrier():
        qdist.barrier(dev)

    sampler = ClockSampler(local_rank)
    sampler.start()          # started before the warm-up: nvidia-smi needs a moment to come up
    for _ in range(args.warmup):
        step()
    barrier()
    # the launches of one step (per layer: reset + 7 kernels) are captured once into a CUDA graph and replayed
    run_step, launch_mode = step, "stream"
    if not args.no_graph:
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            graph.replay()
            torch.cuda.synchronize()
            run_step, launch_mode = graph.replay, "cuda graph"
        except Exception as exc:      # capture refused: plain stream launches
            sys.stderr.write(f"bench: graph capture failed ({exc}); launching on the stream\n")
            torch.cuda.synchronize()
    barrier()
    e0 = ev()
    for _ in range(args.steps):
        run_step()
    e1 = ev()
    barrier()
    clocks = sampler.stop()
    # per-stage times from a separate pass with an event pair around every stage (kept out of the timed steps)
    timers = {"thr": ([], []), "quant": ([], []), "dec": ([], [])}
    for _ in range(min(args.steps, 3)):
        step(timers)
    torch.cuda.synchronize()
    ms_total, _ = qdist.aggregate(e0.elapsed_time(e1), 1.0, dev)     # slowest rank
    ms_step = ms_total / args.steps
    stage_ms = {k: sum(a.elapsed_time(b) for a, b in zip(*v)) / len(v[0]) for k, v in timers.items()}

    st = qaq.qaq_cache_stats(layers[0]["cache"])
    assert st.device_status == 0
    ab = algorithmic_bytes(wl, st)
    step_bytes = L * (ab["thresholds"] + ab["quantize"] + ab["decode"])
    value = world * step_bytes / (ms_step * 1e-3) / 1e9
    quant_gbs = ab["quantize"] / (stage_ms["quant"] * 1e-3) / 1e9
    dec_gbs = ab["decode"] / (stage_ms["dec"] * 1e-3) / 1e9
    thr_gbs = ab["thresholds"] / (stage_ms["thr"] * 1e-3) / 1e9

    counters, cnote = load_counters() if args.workload == "C3" else (None, "counters are kept for the C3 layer shape only")

    def traffic(*keys):
        return None if counters is None or any(k not in counters["kernels"] for k in keys) else round(sum(counters["kernels"][k]["dram_bytes"] for k in keys))

    def instr(*keys):
        return None if counters is None or any(k not in counters["kernels"] for k in keys) else sum(counters["kernels"][k]["warp_instr"] for k in keys)

    out = {
        "metric": METRIC, "value": round(value, 2), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_step, 4), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_of(wl, (sS, sX, hyper_qn)),
        "run": {"mean_bits": [round(st.code_bytes[0] * 8 / (BH * T * D), 3), round(st.code_bytes[1] * 8 / (BH * T * D), 3)],
                "cr_paper": round(st.cr_paper, 3), "cr_total": round(st.cr_total, 3), "hyper_source": hyper_source,
                "qnorm2_quantile_of_this_run": round(qn_measured, 4),
                "l2": "each layer's inputs (>0.5 GB) and packed cache exceed L2; no flush needed",
                "per_rank": "own batch, no collective", "launch": launch_mode, "streams": args.streams,
                "stage_timing": "event pair around every stage in a separate single-stream pass after the timed steps"},
        "quant_plus_decode": {"ms_per_layer": round(stage_ms["quant"] + stage_ms["dec"], 4),
                              "gbs": round((ab["quantize"] + ab["decode"]) / ((stage_ms["quant"] + stage_ms["dec"]) * 1e-3) / 1e9, 1),
                              "note": "the step's value also counts the threshold pass (one more read of K and V)"},
        "stages": {
            "thresholds": {"ms_per_layer": round(stage_ms["thr"], 4), "gbs": round(thr_gbs, 1), "frac_of_hbm": round(thr_gbs / peak, 3)},
            "quantize": {"ms_per_layer": round(stage_ms["quant"], 4), "gbs": round(quant_gbs, 1), "frac_of_hbm": round(quant_gbs / peak, 3),
                         "fp16_input_gbs": round(ab["fp16"] / (stage_ms["quant"] * 1e-3) / 1e9, 1)},
            "decode": {"ms_per_layer": round(stage_ms["dec"], 4), "gbs": round(dec_gbs, 1), "frac_of_hbm": round(dec_gbs / peak, 3),
                       "cached_tokens_per_s": round(wl.batch * T / (stage_ms["dec"] * 1e-3), 1),
                       "generated_tokens_per_s": round(wl.batch / (L * stage_ms["dec"] * 1e-3), 2)},
        },
        "roofline": {"kernel": "quant_kernel, keys launch + values launch (fused select + outlier split + quantize + pack)", "bound": "hbm",
                     "achieved": round(quant_gbs, 1), "peak": peak, "unit": "GB/s", "frac": round(quant_gbs / peak, 3),
                     "traffic": traffic("quant_keys", "quant_values"), "traffic_note": cnote, "peak_kind": peak_kind, "bytes_per_launch": ab["quantize"]},
        "roofline_decode": {"kernel": "decode_kernel (+ merge)", "bound": "hbm", "achieved": round(dec_gbs, 1), "peak": peak,
                            "unit": "GB/s", "frac": round(dec_gbs / peak, 3), "traffic": traffic("decode"), "traffic_note": cnote, "peak_kind": peak_kind,
                            "bytes_per_launch": ab["decode"]},
        "roofline_issue": {"quant_kernel": issue_roofline(instr("quant_keys", "quant_values"), stage_ms["quant"] * 1e-3, clocks.get("sm_mhz")),
                           "decode_kernel": issue_roofline(instr("decode"), stage_ms["dec"] * 1e-3, clocks.get("sm_mhz"))},
        "gpu_launches": args.steps * L * 7,   # thresholds 3 (sample, scan, select), quantize 2 (keys, values), decode 2 (+ merge)
        "clocks": clocks,
    }

    # ---- end to end through the host-buffer C-ABI entry points (pinned host memory, copies in the timed region)
    if not args.no_e2e:
        Ly = layers[0]
        pin = lambda t: t.cpu().contiguous().pin_memory()
        hK, hV, hq, hr, hn, ht = pin(Ly["K"]), pin(Ly["V"]), pin(Ly["q"]), pin(Ly["ring"]), pin(Ly["nv"]), pin(Ly["thr"])
        hout = torch.empty((BH, D), dtype=torch.float32).pin_memory()
        n_e2e = max(1, min(args.steps, 2))

        def e2e_step():
            for Lz in layers:      # every layer gets the bytes of a full layer from the host
                Lz["cache"].reset()
                qaq.qaq_quantize_append_host(Lz["cache"], hK, hV, pol, hr, hn, ht)
                qaq.qaq_decode_attention_host(Lz["cache"], hq, scale, hout)
        e2e_step()
        barrier()
        a = ev()
        for _ in range(n_e2e):
            e2e_step()
        b = ev()
        barrier()
        ms_e2e, _ = qdist.aggregate(a.elapsed_time(b) / n_e2e, 1.0, dev)
        h2d = L * (hK.numel() * 2 * 2 + hr.numel() * 4 + hn.numel() + ht.numel() * 4 + hq.numel() * 2)
        e2e_bytes = L * (ab["quantize"] + ab["decode"])
        out["e2e"] = {"value": round(world * e2e_bytes / (ms_e2e * 1e-3) / 1e9, 2), "unit": "GB/s",
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": L * hout.numel() * 4, "ms_per_step": round(ms_e2e, 3),
                      "steps": n_e2e, "note": "quantize_append_host + decode_attention_host per layer; thresholds resident"}

    # ---- CPU oracle beside it (rank 0, N = 1 only): a bounded sample of the same workload
    # ---- the other 7B-shaped configurations, for context (rank 0, one GPU): one layer at batch 1 (launch-latency
    # regime) and the long-context cache (values of tokens beyond the prefill stay at 8 bits: no score seen yet)
    if rank == 0 and world == 1 and not args.no_extras:
        out["extras"] = extras(qaq, dev, peak, args.extras, clocks.get("sm_mhz"))

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(wl, (sS, sX, hyper_qn))

    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


def _time_us(fn, reps):
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        fn()
    b.record(); torch.cuda.synchronize()
    return a.elapsed_time(b) * 1e3 / reps


def extras(qaq, dev, peak, only="", sm_mhz=None):
    from paper_2403_04643_b200.calibrate import frozen
    res = {}
    c3 = synth.scaled(synth.CONFIGS["C3"], layers=1)
    # (name, workload, tokens, prefill, frozen hyper-parameters (hyper.json) or None, constant width or None)
    points = (("C2_layer_batch1", synth.CONFIGS["C2"], 4096, 4096, "C2", None),
              ("C5_long_context", synth.CONFIGS["C5"], 131072, 32768, "C5", None),
              # low widths, the stress case for instruction issue (compression ratio near the paper's)
              ("C3_layer_low_widths", c3, c3.tokens, c3.tokens, "C3_low", None),
              # the comparison codec of Section 5.2: one width for every token, outliers kept apart as before
              ("C3_layer_uniform4_with_outliers", c3, c3.tokens, c3.tokens, None, 4))
    for name, wl, T, prefill, hname, uniform in points:
        if only and not name.startswith(only):
            continue
        D, BH, W = wl.head_dim, wl.bh, wl.window
        wlx = synth.scaled(wl, tokens=T, grow_to=0)
        K, V = synth.make_kv(wlx, 0, device=dev)
        q = synth.make_query(wlx, 0, device=dev)
        ring, nv = synth.make_score_ring(wlx, 0, device=dev)
        nv[:, :, prefill:] = 0                       # tokens appended after the prefill have no score yet
        cfg = qaq.make_config(wl.batch, wl.heads, D, T + 64, wl.bits_min, wl.bits_max, W, wl.alpha)
        thr = qaq.qaq_outlier_thresholds(cfg, K[:, :, :prefill], V[:, :, :prefill])
        pol, given = None, {}
        if uniform is None:
            pol = qaq.qaq_policy_from_hyper(*frozen(hname), prefill)
        else:
            bits = torch.full((BH, T), uniform, dtype=torch.uint8, device=dev)
            given = {"bitsK": bits, "bitsV": bits}
        cache = qaq.Cache(cfg)
        outb = torch.empty((BH, D), dtype=torch.float32, device=dev)
        scale = 1.0 / math.sqrt(D)

        def fill():
            cache.reset()
            if uniform is None:
                qaq.qaq_quantize_append(cache, K, V, thr, policy=pol, ring=ring, nvalid=nv)
            else:
                qaq.qaq_quantize_append(cache, K, V, thr, **given)
        us_q = _time_us(fill, 5)
        us_d = _time_us(lambda: qaq.qaq_decode_attention(cache, q, scale, out=outb), 20)
        st = qaq.qaq_cache_stats(cache)
        ab = algorithmic_bytes(wlx, st)
        if uniform is not None:     # given widths: two width bytes per token-head are read instead of the score window
            ab["quantize"] += (2 - (4 * W + 1)) * BH * T
        # one-token append + decode, the streaming step
        k1, v1 = K[:, :, :1].contiguous(), V[:, :, :1].contiguous()
        r1, n1 = ring[:, :, :, :1].contiguous(), torch.zeros((wl.batch, wl.heads, 1), dtype=torch.uint8, device=dev)
        t_now = cache.tokens
        reps = min(32, cfg.max_tokens - t_now)

        b1 = torch.full((BH, 1), uniform or 0, dtype=torch.uint8, device=dev)

        def stream():
            if uniform is None:
                qaq.qaq_quantize_append(cache, k1, v1, thr, policy=pol, ring=r1, nvalid=n1)
            else:
                qaq.qaq_quantize_append(cache, k1, v1, thr, bitsK=b1, bitsV=b1)
            qaq.qaq_decode_attention(cache, q, scale, out=outb)
        torch.cuda.synchronize()
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            stream()
        b.record(); torch.cuda.synchronize()
        us_s = a.elapsed_time(b) * 1e3 / reps
        # the same step with the token count in device memory, captured once in a CUDA graph and replayed
        qaq.qaq_stream_begin(cache)

        def stream_counted():
            if uniform is None:
                qaq.qaq_stream_append(cache, k1, v1, thr, policy=pol, score_col=r1, nvalid=n1)
            else:
                qaq.qaq_stream_append(cache, k1, v1, thr, bitK=b1, bitV=b1)
            qaq.qaq_stream_decode(cache, q, scale, outb)
        stream_counted()                      # loads the kernels before the capture
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            stream_counted()
        reps_g = min(24, cfg.max_tokens - t_now - reps - 1)
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps_g - 3):
            graph.replay()
        b.record(); torch.cuda.synchronize()
        us_g = a.elapsed_time(b) * 1e3 / (reps_g - 3)
        assert qaq.qaq_stream_end(cache) == t_now + reps + 1 + reps_g
        del graph
        res[name] = {"tokens": T, "bh": BH, "quantize_us": round(us_q, 1), "quantize_gbs": round(ab["quantize"] / us_q / 1e3, 1),
                     "quantize_frac_of_hbm": round(ab["quantize"] / us_q / 1e3 / peak, 3),
                     "decode_us": round(us_d, 1), "decode_gbs": round(ab["decode"] / us_d / 1e3, 1),
                     "decode_frac_of_hbm": round(ab["decode"] / us_d / 1e3 / peak, 3),
                     "cached_tokens_per_s": round(wl.batch * T / (us_d * 1e-6), 1),
                     "append1_plus_decode_us": round(us_s, 1), "append1_plus_decode_graph_replay_us": round(us_g, 1),
                     "mean_bits": [round(st.code_bytes[0] * 8 / (BH * T * D), 2), round(st.code_bytes[1] * 8 / (BH * T * D), 2)],
                     "cr_paper": round(st.cr_paper, 3)}
        if name == "C3_layer_low_widths":      # fewer bytes, the same instructions: the issue ceiling is the one that binds
            res[name]["note"] = "fewer bytes per token, the same per-token work: the instruction-issue ceiling binds"
        if name == "C3_layer_uniform4_with_outliers":
            # batched decode (Section 4.2, integration): n_q queries per (b,h) in one call, against n_q single calls
            mq = {}
            for n_q in (1, 4, 8):
                Qm = torch.randn((BH, n_q, D), device=dev, dtype=torch.float32).to(torch.float16)
                om = torch.empty((BH, n_q, D), dtype=torch.float32, device=dev)
                us_m = _time_us(lambda: qaq.qaq_decode_attention_multi(cache, Qm, scale, out=om), 10)
                mq[f"n_q={n_q}"] = {"us": round(us_m, 1), "us_per_query": round(us_m / n_q, 1),
                                    "packed_bytes_per_s_over_hbm_peak": round(ab["decode"] * ((n_q + 3) // 4) / us_m / 1e3 / peak, 3),
                                    "queries_x_cached_tokens_per_s": round(n_q * wl.batch * T / (us_m * 1e-6), 1)}
            mq["single_query_call_us"] = round(us_d, 1)
            res["C3_layer_multi_query_decode"] = mq
            # the score window after a prefill (Section 4.2): rows of the last `window` queries on the fp16 keys
            Qw = torch.randn((BH, W, D), device=dev, dtype=torch.float32).to(torch.float16)
            us_w = _time_us(lambda: qaq.qaq_prefill_window(cfg, Qw, K, scale), 10)
            moved = BH * T * (2 * D + 4 * W + 1)               # K once, the ring once (one-pass kernel up to 4096 tokens)
            res["C3_layer_prefill_window"] = {"rows": W, "us": round(us_w, 1), "bytes": int(moved),
                                              "gbs": round(moved / us_w / 1e3, 1), "frac_of_hbm": round(moved / us_w / 1e3 / peak, 3)}
        if name == "C3_layer_low_widths":
            # the per-step lowering of widths (Section 4.2): a cache filled at mean widths (4, 3) is taken down to the
            # widths of this point's looser budgets, in place; one call does the work, a repeat finds nothing to lower
            pol43 = qaq.qaq_policy_from_hyper(*frozen("C3"), T)
            cache.reset()
            qaq.qaq_quantize_append(cache, K, V, thr, policy=pol43, ring=ring, nvalid=nv)
            qaq.qaq_requantize_down(cache, policy=pol43, ring=ring, nvalid=nv)     # warm-up: same widths, nothing changes
            st0 = qaq.qaq_cache_stats(cache)
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            torch.cuda.synchronize()
            ev[0].record()
            qaq.qaq_requantize_down(cache, policy=pol, ring=ring, nvalid=nv)
            ev[1].record()
            qaq.qaq_requantize_down(cache, policy=pol, ring=ring, nvalid=nv)
            ev[2].record(); torch.cuda.synchronize()
            st1 = qaq.qaq_cache_stats(cache)
            moved = sum(st0.code_bytes) + sum(st1.code_bytes) + BH * T * (2 * 5 + 2 + 4 * W + 1)
            us_r = ev[0].elapsed_time(ev[1]) * 1e3
            res["C3_layer_requantize_down"] = {
                "from_mean_bits": [round(st0.code_bytes[x] * 8 / (BH * T * D), 2) for x in range(2)],
                "to_mean_bits": [round(st1.code_bytes[x] * 8 / (BH * T * D), 2) for x in range(2)],
                "requantize_us": round(us_r, 1), "bytes": int(moved), "gbs": round(moved / us_r / 1e3, 1),
                "frac_of_hbm": round(moved / us_r / 1e3 / peak, 3),
                "repeat_nothing_to_lower_us": round(ev[1].elapsed_time(ev[2]) * 1e3, 1),
                "decode_after_us": round(_time_us(lambda: qaq.qaq_decode_attention(cache, q, scale, out=outb), 20), 1)}
            # and back up to (4, 3) from the unquantized copy: in device memory, then in pinned host memory that the
            # kernel reads through the bus (only the rows of raised tokens)
            big = qaq.make_config(wl.batch, wl.heads, D, 2 * T, wl.bits_min, wl.bits_max, W, wl.alpha)   # room for tiles that move
            up = {}
            for where in ("device", "pinned_host"):
                c2 = qaq.Cache(big)
                qaq.qaq_quantize_append(c2, K, V, thr, policy=pol, ring=ring, nvalid=nv)
                Ks, Vs = (K, V) if where == "device" else (K.cpu().pin_memory(), V.cpu().pin_memory())
                torch.cuda.synchronize()
                e = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
                e[0].record()
                qaq.qaq_requantize(c2, Ks, Vs, thr, policy=pol43, ring=ring, nvalid=nv)
                e[1].record(); torch.cuda.synchronize()
                stu = qaq.qaq_cache_stats(c2)
                up[where + "_us"] = round(e[0].elapsed_time(e[1]) * 1e3, 1)
                up["to_mean_bits"] = [round(stu.code_bytes[x] * 8 / (BH * T * D), 2) for x in range(2)]
                up["device_status"] = int(stu.device_status)
                del c2, Ks, Vs
            res["C3_layer_requantize_up"] = up
        del cache, K, V, ring
        torch.cuda.empty_cache()
    if not only or "C2_generation_loop".startswith(only):
        res["C2_generation_loop"] = generation_loop_c2(qaq, dev)
    if not only or "C5_stream_all_steps".startswith(only):
        res["C5_stream_all_steps"] = stream_c5(qaq, dev)
    return res


def generation_loop_c2(qaq, dev, steps=256):
    """The per-step loop of Section 4.2 ("Integration in text generation process") on one 7B-shaped layer at batch 1:
    append the new token, decode with the normalised score row written out, put that row into the window (the
    caller's ring: plain tensor copies), then lower the widths of all cached tokens to what the rules give with the
    new window (qaq_requantize_down)."""
    from paper_2403_04643_b200.calibrate import frozen
    wl = synth.CONFIGS["C2"]
    T0, D, BH, W = wl.tokens, wl.head_dim, wl.bh, wl.window
    T1 = T0 + steps
    wlx = synth.scaled(wl, tokens=T1)
    K, V = synth.make_kv(wlx, 0, device=dev)
    q = synth.make_query(wlx, 0, device=dev)
    ring0, nv0 = synth.make_score_ring(wl, 0, device=dev)
    ring = torch.zeros((wl.batch, wl.heads, W, T1), dtype=torch.float32, device=dev)
    nvalid = torch.zeros((wl.batch, wl.heads, T1), dtype=torch.uint8, device=dev)
    ring[:, :, :, :T0] = ring0; nvalid[:, :, :T0] = nv0
    # room for tiles that move: a value tile whose widths are lowered can need more padding of its groups than before
    cfg = qaq.make_config(wl.batch, wl.heads, D, 2 * T1, wl.bits_min, wl.bits_max, W, wl.alpha)
    thr = qaq.qaq_outlier_thresholds(cfg, K[:, :, :T0], V[:, :, :T0])
    hy = frozen("C2")
    cache = qaq.Cache(cfg)
    qaq.qaq_quantize_append(cache, K[:, :, :T0], V[:, :, :T0], thr, policy=qaq.qaq_policy_from_hyper(*hy, T0), ring=ring0, nvalid=nv0)
    st0 = qaq.qaq_cache_stats(cache)
    outb = torch.empty((BH, D), dtype=torch.float32, device=dev)
    r1 = torch.zeros((wl.batch, wl.heads, W, 1), dtype=torch.float32, device=dev)
    n1 = torch.zeros((wl.batch, wl.heads, 1), dtype=torch.uint8, device=dev)
    scale = 1.0 / math.sqrt(D)

    def one(t):
        pol = qaq.qaq_policy_from_hyper(*hy, t + 1)
        qaq.qaq_quantize_append(cache, K[:, :, t:t + 1], V[:, :, t:t + 1], thr, policy=pol, ring=r1, nvalid=n1)
        qaq.qaq_decode_attention(cache, q, scale, out=outb, scores_out=scores_view(t + 1))
        ring[:, :, t % W, :t + 1] = scores_view(t + 1).view(wl.batch, wl.heads, t + 1)
        nvalid[:, :, :t + 1] = torch.clamp(nvalid[:, :, :t + 1] + 1, max=W)
        qaq.qaq_requantize_down(cache, policy=pol, ring=ring, nvalid=nvalid)
        if (t - T0) % 64 == 63:
            qaq.qaq_cache_compact(cache)      # closes the gaps moved tiles leave in the pools

    sbuf = torch.empty((BH * T1,), dtype=torch.float32, device=dev)

    def scores_view(n):
        return sbuf[:BH * n].view(BH, n)

    for t in range(T0, T0 + 8):
        one(t)
    torch.cuda.synchronize()
    a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
    a.record()
    for t in range(T0 + 8, T1):
        one(t)
    b.record(); torch.cuda.synchronize()
    st1 = qaq.qaq_cache_stats(cache)
    n = T1 - T0 - 8
    mb = lambda st, x: round(st.code_bytes[x] * 8 / (BH * st.tokens * D), 2)
    return {"steps": n, "us_per_step": round(a.elapsed_time(b) * 1e3 / n, 1), "tokens_at_end": int(st1.tokens),
            "mean_bits_after_prefill": [mb(st0, 0), mb(st0, 1)], "mean_bits_at_end": [mb(st1, 0), mb(st1, 1)],
            "cr_paper_at_end": round(st1.cr_paper, 3), "device_status": int(st1.device_status),
            "note": "append 1 + decode with score row + window update (tensor copies) + qaq_requantize_down over the whole cache, per step"}


def stream_c5(qaq, dev):
    """The long-context configuration as stated: a 32768-token prefill grown to 131072 tokens by one-token appends,
    every step quantizing the new token and running packed decode attention (all 98304 steps, launched one by one)."""
    from paper_2403_04643_b200.calibrate import frozen
    wl = synth.CONFIGS["C5"]
    T0, T1 = wl.tokens, wl.grow_to
    wlx = synth.scaled(wl, tokens=T1, grow_to=0)
    D, BH, W = wl.head_dim, wl.bh, wl.window
    K, V = synth.make_kv(wlx, 0, device=dev)
    q = synth.make_query(wlx, 0, device=dev)
    ring, nv = synth.make_score_ring(synth.scaled(wl, grow_to=0), 0, device=dev)
    cfg = qaq.make_config(wl.batch, wl.heads, D, T1, wl.bits_min, wl.bits_max, W, wl.alpha)
    thr = qaq.qaq_outlier_thresholds(cfg, K[:, :, :T0], V[:, :, :T0])
    pol = qaq.qaq_policy_from_hyper(*frozen("C5"), T0)
    cache = qaq.Cache(cfg)
    qaq.qaq_quantize_append(cache, K[:, :, :T0], V[:, :, :T0], thr, policy=pol, ring=ring, nvalid=nv)
    r1 = torch.zeros((wl.batch, wl.heads, W, 1), dtype=torch.float32, device=dev)
    n1 = torch.zeros((wl.batch, wl.heads, 1), dtype=torch.uint8, device=dev)
    outb = torch.empty((BH, D), dtype=torch.float32, device=dev)
    scale = 1.0 / math.sqrt(D)
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    torch.cuda.synchronize()
    a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
    a.record()
    for t in range(T0, T1):
        qaq.qaq_quantize_append(cache, K[:, :, t:t + 1], V[:, :, t:t + 1], thr, policy=pol, ring=r1, nvalid=n1)
        qaq.qaq_decode_attention(cache, q, scale, out=outb)
    b.record(); torch.cuda.synchronize()
    sec = a.elapsed_time(b) * 1e-3
    st = qaq.qaq_cache_stats(cache)
    res = {"steps": T1 - T0, "seconds": round(sec, 2), "us_per_step": round(sec / (T1 - T0) * 1e6, 1),
           "generated_tokens_per_s": round(wl.batch * (T1 - T0) / sec, 1), "final_tokens": int(st.tokens),
           "device_status": int(st.device_status),
           "note": "host-launched steps (one append launch, decode + merge per step); values of appended tokens stay at 8 bits"}
    # the same run with the token count in device memory: one captured append + decode pair replayed 98304 times, the
    # new token's rows copied into the captured buffers before every replay
    cache.reset()
    qaq.qaq_quantize_append(cache, K[:, :, :T0], V[:, :, :T0], thr, policy=pol, ring=ring, nvalid=nv)
    k1 = torch.empty((wl.batch, wl.heads, 1, D), dtype=torch.float16, device=dev)
    v1 = torch.empty_like(k1)
    warm = qaq.Cache(qaq.make_config(wl.batch, wl.heads, D, 64, wl.bits_min, wl.bits_max, W, wl.alpha))
    k1.zero_(); v1.zero_()
    qaq.qaq_stream_begin(warm)                 # one eager step on a scratch cache loads the kernels before the capture
    qaq.qaq_stream_append(warm, k1, v1, thr, policy=pol, score_col=r1, nvalid=n1)
    qaq.qaq_stream_decode(warm, q, scale, outb)
    qaq.qaq_stream_end(warm)
    warm.close()
    cache.workspace()
    qaq.qaq_stream_begin(cache)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        qaq.qaq_stream_append(cache, k1, v1, thr, policy=pol, score_col=r1, nvalid=n1)
        qaq.qaq_stream_decode(cache, q, scale, outb)
    a.record()
    for t in range(T0, T1):
        k1.copy_(K[:, :, t:t + 1]); v1.copy_(V[:, :, t:t + 1])
        graph.replay()
    b.record(); torch.cuda.synchronize()
    sec_g = a.elapsed_time(b) * 1e-3
    final = qaq.qaq_stream_end(cache)
    st = qaq.qaq_cache_stats(cache)
    res["graph_replay"] = {"seconds": round(sec_g, 2), "us_per_step": round(sec_g / (T1 - T0) * 1e6, 1),
                           "generated_tokens_per_s": round(wl.batch * (T1 - T0) / sec_g, 1), "final_tokens": int(final),
                           "device_status": int(st.device_status)}
    res["clocks"] = sampler.stop()
    return res


def cpu_baseline(wl, hyper, budget_s=15.0):
    cores = os.cpu_count() or 1
    n_bh = min(wl.bh, 16 * cores)
    run = oracle_sample(wl, hyper, n_bh, cores, "cpu")
    dt, r = run()
    reps = 1
    total = dt
    while total + dt < budget_s and reps < 12:
        d2, r = run()
        total += d2
        reps += 1
    sec = total / reps
    gbs = n_bh * wl.tokens * per_th_bytes(wl) / sec / 1e9
    return {"value": round(gbs, 4), "unit": "GB/s", "cores": int(r.threads), "kind": "oracle",
            "sample": f"{n_bh} of {wl.bh} (b,h) of layer 0 ({wl.tokens} tokens each): thresholds + select + quantize + decode, "
                      f"{reps} repetition(s), {sec:.2f} s each; bytes at nominal widths (4,3)",
            "cached_tokens_per_s": round(n_bh * wl.tokens / wl.heads / sec, 1)}


def reference_arm(args, wl, hyper):
    """The oracle as the reference arm: every step is a bounded sample of the workload, on the same configuration
    (frozen hyper-parameters) as the GPU arm."""
    cores = os.cpu_count() or 1
    if hyper is None:
        hyper = (0.002, 0.01, 1.16)
    n_bh = min(wl.bh, 16 * cores)
    run = oracle_sample(wl, hyper, n_bh, cores, "cpu")
    for _ in range(args.warmup):
        run()
    ts = []
    threads = cores
    for _ in range(max(1, args.steps)):
        dt, r = run()
        ts.append(dt)
        threads = r.threads
    sec = sum(ts) / len(ts)
    gbs = n_bh * wl.tokens * per_th_bytes(wl) / sec / 1e9
    sample = f"{n_bh} of {wl.bh} (b,h) of one layer per step ({wl.tokens} tokens each), {len(ts)} timed step(s)"
    out = {"impl": "reference", "metric": METRIC, "value": round(gbs, 4), "unit": "GB/s", "n_gpus": args.gpus,
           "steps": len(ts), "warmup": args.warmup, "ms_per_step": round(sec * 1e3, 2), "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
           "config": config_of(wl, hyper),
           "cpu_baseline": {"value": round(gbs, 4), "unit": "GB/s", "cores": int(threads), "kind": "oracle", "sample": sample},
           "e2e": {"value": round(gbs, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))
    return 0


if __name__ == "__main__":
    sys.exit(main())
