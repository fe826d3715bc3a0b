#!/usr/bin/env python
"""Benchmark of the MARche decoding hot path: 64-step synthetic MAR-L-shaped generation.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--config mar_l] [--ratio 0.1] [--blocks L] [--batch B] [--no-extras]

One "step" of this benchmark is one whole T-step generation of a batch (B rows = B/2
images with classifier-free-guidance pairs): a full step that fills the K/V cache and
T-1 cache-aware steps, all through the C ABI of libmarche.  Only the transformer stack
is timed; the sampler and the VAE are outside the hot path.  Rank 0 prints ONE JSON line.

The path does not shard (one GPU holds a model replica and its own samples; there is no
exchange step), so N > 1 runs N independent replicas and reports the aggregate
("scaling": "weak").

--impl reference times the CPU oracle (the deliberately plain NumPy restatement of the
method) on a bounded sample of the same workload on this machine's host cores.
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

import synth

# Fallback roofline denominators (an earlier measurement on this machine), used only when
# MEASURED_PEAKS.json is absent.
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_dram_traffic.txt")


def load_ncu_traffic():
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel
    classes, as written from an ncu capture by `bench.py --write-traffic <ncu raw csv>`:
    lines `class bytes_per_launch launches`.  {} when the file is absent."""
    out = {}
    if os.path.exists(TRAFFIC_FILE):
        for ln in open(TRAFFIC_FILE):
            f = ln.split()
            if len(f) >= 2 and not ln.startswith("#"):
                out[f[0]] = float(f[1])
    return out


def write_ncu_traffic(csv_paths):
    """Reads `ncu -i <report> --page raw --csv` outputs (comma-separated paths) and writes the mean DRAM
    bytes per launch of the GEMM and attention kernels to profiles/ncu_dram_traffic.txt."""
    import csv
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    acc = {}
    for csv_path in csv_paths.split(","):
        rows = list(csv.reader(open(csv_path)))
        hdr = next(r for r in rows if "Kernel Name" in r)
        units = rows[rows.index(hdr) + 1]
        i_name = hdr.index("Kernel Name")
        i_rd, i_wr = hdr.index("dram__bytes_read.sum"), hdr.index("dram__bytes_write.sum")
        for r in rows[rows.index(hdr) + 2:]:
            if len(r) <= max(i_rd, i_wr):
                continue
            name = r[i_name]
            cls = "gemm" if "gemm_tcgen05" in name else ("attention" if "attention_mma" in name and ", 0>" in name else
                                                         ("attention_tc_stream" if "attention_tc_stream" in name else None))
            if cls is None:
                continue
            b = float(r[i_rd].replace(",", "")) * scale[units[i_rd]] + float(r[i_wr].replace(",", "")) * scale[units[i_wr]]
            acc.setdefault(cls, []).append(b)
    with open(TRAFFIC_FILE, "w") as f:
        f.write("# mean dram__bytes_read.sum + dram__bytes_write.sum per launch, from ncu --set full captures of\n"
                "# 4-block slices of the benchmark workloads (see the *.md summaries beside this file for the commands)\n")
        f.write("# class bytes_per_launch launches\n")
        for cls, v in sorted(acc.items()):
            f.write("%s %.0f %d\n" % (cls, float(np.mean(v)), len(v)))
    print(open(TRAFFIC_FILE).read())


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ----------------------------------------------------------------------------- replicas (N > 1)
def max_over_ranks(value: float, device="cuda") -> float:
    """The slowest rank's time: with N independent replicas the job is as slow as its slowest GPU."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_images_per_s(n_images_per_rank: int, ms_max: float, world: int) -> float:
    """Whole-job throughput of `world` replicas that each generate n_images_per_rank images."""
    return world * n_images_per_rank / (ms_max * 1e-3)


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        self.lines = []
        self.idx = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "power_w_max": float(max(power)), "samples": len(sm)}


# ----------------------------------------------------------------------------- workload bookkeeping
def schedule(cfg, ratio):
    """Per step: (#G, nA, k) of the cache-aware generation (k selected at the step for the next)."""
    counts = synth.mask_schedule(cfg.n_img, cfg.T)
    want = int(np.floor(ratio * cfg.S + 0.5))
    out, k_prev = [], 0
    for t, g in enumerate(counts):
        nxt = counts[t + 1] if t + 1 < cfg.T else 0
        nA = cfg.S if t == 0 else g + counts[t - 1] + k_prev
        k = min(want, cfg.S - g - nxt)
        out.append((g, nA, k))
        k_prev = k
    return out


def algorithmic_work(cfg, sched):
    """Algorithmic flops / bytes for each kernel class over the given steps (16-bit operands, fp32
    residual): per step and block, K1 reads M*D*4 and writes M*D*2 (twice per block, plus the compact
    fp32 copy at block 0); K2 does 2*M*(4*D*D + 2*D*F) flops; K5 moves 2*M*D*2 bytes in and out; K3 reads
    K and V of all S tokens plus Q and writes O; K4 reads the score partials and the mask."""
    B, S, D, F, L, H = cfg.B, cfg.S, cfg.D, cfg.F, cfg.L, cfg.H
    w = {"gemm_flops": 0.0, "attention_bytes": 0.0, "attention_flops": 0.0, "gather_layernorm_bytes": 0.0,
         "scatter_kv_bytes": 0.0, "scatter_rows_bytes": 0.0, "topk_bytes": 0.0}
    w["gemm_split"] = {"gemm_qkv": 3.0 * D * D, "gemm_out_proj": 1.0 * D * D, "gemm_fc1_gelu": 1.0 * D * F,
                       "gemm_fc2": 1.0 * D * F}
    for g, nA, k in sched:
        M = B * nA
        w["gemm_flops"] += 2.0 * M * (4 * D * D + 2 * D * F) * L
        w["attention_bytes"] += (2.0 * B * S * D * 2 + 2.0 * M * D * 2) * L + B * H * S * 4
        w["attention_flops"] += 4.0 * B * nA * S * D * L
        w["gather_layernorm_bytes"] += 2 * (M * D * 4 + M * D * 2) * L + M * D * 4
        w["scatter_kv_bytes"] += 4.0 * M * D * 2 * L
        w["scatter_rows_bytes"] += 2.0 * M * D * 4 + 2.0 * B * g * D * 4
        w["topk_bytes"] += B * H * S * 4 + B * S * 5 + B * k * 4
    return w


GEMM_CLASSES = ("gemm_qkv", "gemm_out_proj", "gemm_fc1_gelu", "gemm_fc2")


def kernel_table(prof, work, peaks, attention_bound):
    """Per-kernel-class roofline rows from one profile (class -> (ms, launches)) and the
    algorithmic work of the same steps."""
    total_ms = sum(v[0] for v in prof.values())
    rows = []

    def add(name, bound, amount, ms, n, peak, unit):
        if n == 0 or ms <= 0:
            return
        ach = amount / (ms * 1e-3) / (1e12 if unit == "TFLOP/s" else 1e9)
        rows.append({"kernel": name, "bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                     "launches": n, "ms": ms, "us_per_launch": 1e3 * ms / n, "share": ms / total_ms})

    add("gemm_tcgen05 (qkv, out, fc1, fc2)", "tensor", work["gemm_flops"], sum(prof[c][0] for c in GEMM_CLASSES),
        sum(prof[c][1] for c in GEMM_CLASSES), peaks["bf16_tflops_sustained"], "TFLOP/s")
    # the same row split by projection (flops in proportion 3 D^2 : D^2 : D F : D F)
    if rows and "gemm_split" in work:
        tot = sum(work["gemm_split"].values())
        rows[-1]["by_projection"] = {
            c: {"us_per_launch": 1e3 * prof[c][0] / prof[c][1],
                "frac": work["gemm_flops"] * work["gemm_split"][c] / tot / (prof[c][0] * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"]}
            for c in GEMM_CLASSES if prof[c][1]}
    if attention_bound == "hbm":
        add("attention", "hbm", work["attention_bytes"], *prof["attention"], peaks["hbm_gbs"], "GB/s")
    else:
        add("attention", "tensor", work["attention_flops"], *prof["attention"], peaks["bf16_tflops_sustained"], "TFLOP/s")
    add("gather_layernorm", "hbm", work["gather_layernorm_bytes"], *prof["gather_layernorm"], peaks["hbm_gbs"], "GB/s")
    add("scatter_kv", "hbm", work["scatter_kv_bytes"], *prof["scatter_kv"], peaks["hbm_gbs"], "GB/s")
    add("scatter_rows", "hbm", work["scatter_rows_bytes"], *prof["scatter_rows"], peaks["hbm_gbs"], "GB/s")
    add("topk", "hbm", work["topk_bytes"], *prof["topk"], peaks["hbm_gbs"], "GB/s")
    rows.sort(key=lambda r: -r["ms"])
    return rows


# ----------------------------------------------------------------------------- reference arm (CPU oracle)
def oracle_sample(cfg, ratio, n_cache_steps=2):
    """Times the oracle on one CFG pair (2 of the B rows): 1 full step + n cache-aware steps,
    and extrapolates to a T-step generation.  Returns (images_per_s, seconds_per_generation, dict)."""
    from oracle import marche_oracle as orc
    pair = cfg.replace(B=2)
    blocks = synth.make_weights(cfg)
    hidden = synth.make_hidden(cfg, batch=2)
    orders = synth.generation_orders(cfg)
    sets = [g[[0, cfg.B // 2]] if cfg.cfg_pairs else g[:2] for g in synth.new_token_sets(cfg, orders)]
    kw = dict(n_heads=cfg.H, score_layer=cfg.score_layer, ln_eps=cfg.ln_eps)
    cache = orc.KVCache(cfg.L, 2, cfg.S, cfg.D)
    out = np.zeros_like(hidden)
    t0 = time.perf_counter()
    _, R = orc.full_step(blocks, hidden, cache, sets[0], sets[1], ratio, out, **kw)
    t_full = time.perf_counter() - t0
    t_steps = []
    for t in range(1, 1 + n_cache_steps):
        rows = synth.replacement_rows(cfg, t - 1, sets[t - 1].shape[1], batch=2)
        for b in range(2):
            hidden[b, sets[t - 1][b]] = rows[b]
        A = orc.active_set(sets[t], sets[t - 1], R)
        t0 = time.perf_counter()
        _, R = orc.marche_step(blocks, hidden, cache, A, sets[t], sets[t + 1], ratio, out, **kw)
        t_steps.append(time.perf_counter() - t0)
    t_gen = t_full + (cfg.T - 1) * float(np.mean(t_steps))     # one image (its CFG pair), T steps
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    info = {"kind": "oracle", "cores": int(cores),
            "sample": "one CFG pair (2 of %d rows): 1 full step (%.2f s) + %d cache-aware steps (%.2f s each), "
                      "extrapolated to %d steps" % (cfg.B, t_full, n_cache_steps, float(np.mean(t_steps)), cfg.T)}
    return 1.0 / t_gen, t_gen, info


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    for _ in range(args.warmup):                 # untimed: pages in NumPy / BLAS threads and the weight generator
        oracle_sample(cfg, args.ratio, n_cache_steps=1)
    for _ in range(args.steps):
        ips, t_gen, info = oracle_sample(cfg, args.ratio)
        vals.append((ips, t_gen))
    ips = float(np.mean([v[0] for v in vals]))
    t_gen = float(np.mean([v[1] for v in vals]))
    info = dict(info, value=ips, unit="images/s")
    line = {"impl": "reference", "metric": METRIC, "value": ips, "unit": "images/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_gen * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(cfg, args.ratio), "cpu_baseline": info,
            "e2e": {"value": ips, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


METRIC = "images/s (64-step MAR-L-shaped, bs128)"


def workload_config(cfg, ratio):
    return {"workload": "%s: %d blocks, width %d, %d heads, MLP %d, %d tokens (%d image + %d buffer), batch %d "
                        "(CFG-doubled), %d steps cosine schedule, refresh ratio %g; transformer stack only"
                        % (cfg.name, cfg.L, cfg.D, cfg.H, cfg.F, cfg.S, cfg.n_img, cfg.n_buffer, cfg.B, cfg.T, ratio),
            "config_name": cfg.name, "refresh_ratio": ratio, "l2": "working set (K/V cache + weights) exceeds L2",
            "timed": "T-step generation per bench step"}


# ----------------------------------------------------------------------------- our arm
def run_ours(args, cfg):
    import torch
    import torch.distributed as dist

    from paper_2506_12035_b200.binding import Marche, upload_weights
    from paper_2506_12035_b200.generation import Generation

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks, peak_kind = load_peaks()

    ratio = args.ratio
    blocks = synth.make_weights(cfg)
    m = Marche.from_config(cfg, upload_weights(blocks, cfg.dtype, operand=args.operand))
    del blocks
    hidden0_np = synth.make_hidden(cfg)
    sets = synth.new_token_sets(cfg, synth.generation_orders(cfg))
    rows_np = [synth.replacement_rows(cfg, t, sets[t].shape[1]) for t in range(cfg.T)]
    gen = Generation(m, sets, ratio, [torch.as_tensor(r).cuda() for r in rows_np])
    hidden0 = torch.as_tensor(hidden0_np).cuda()
    sched = schedule(cfg, ratio)
    work = algorithmic_work(cfg, sched)
    n_images = cfg.n_images

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, reps):
        """max-over-ranks device time of `reps` calls of fn, in ms per call."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1)) / reps

    n_dec = args.decode_steps or None
    for _ in range(args.warmup):
        gen.run(hidden0, n_steps=n_dec)
    torch.cuda.synchronize()
    # The timed step: the whole generation recorded once as a CUDA graph and replayed (the kernels, their
    # arguments and their order are exactly those of the stream-launched generation; what goes away is the
    # host's per-launch work).  --stream-launch, or a failed capture, times the stream-launched generation.
    graph, per_replay, launch_mode = None, 0, "stream launches"
    if not args.stream_launch and n_dec is None:
        try:
            l0 = m.launch_count()
            graph = gen.capture(hidden0)
            per_replay = (m.launch_count() - l0) // 2              # one eager generation, one recorded
            for _ in range(2):
                graph.replay()
            torch.cuda.synchronize()
            launch_mode = "one CUDA graph per generation (%d kernel nodes)" % per_replay
        except Exception as exc:
            graph, launch_mode = None, "stream launches (graph capture failed: %s)" % str(exc)[:120]
    step_fn = (lambda: graph.replay()) if graph is not None else (lambda: gen.run(hidden0, n_steps=n_dec))
    clocks = ClockSampler(local)
    clocks.start()
    launches0 = m.launch_count()
    ms_gen = timed(step_fn, args.steps)
    launches = per_replay * args.steps if graph is not None else m.launch_count() - launches0
    clock_info = clocks.stop()
    assert m.device_status() == 0, "a bounded device wait gave up"
    value = aggregate_images_per_s(n_images, ms_gen, world)

    line = {"metric": METRIC, "value": value, "unit": "images/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_gen, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None,
            "dtype": ("%s projections + bf16 attention/cache, fp32 accumulate" % ("fp16" if args.operand == "f16" else "bf16"))
                     if cfg.dtype == "bf16" else "f32", "data": "synthetic",
            "config": dict(workload_config(cfg, ratio), launch=launch_mode), "clocks": clock_info,
            "gpu_launches": int(launches), "ms_per_decoding_step": ms_gen / cfg.T}
    if graph is not None and not args.no_extras:
        ms_stream = timed(lambda: gen.run(hidden0), 2)
        line["stream_launched"] = {"value": aggregate_images_per_s(n_images, ms_stream, world), "unit": "images/s",
                                   "ms_per_step": ms_stream}

    if not args.no_extras:
        # ---- per-kernel-class device time of one more generation (an event in front of every
        # launch; events serialise the launches, so programmatic dependent launch does not overlap
        # here and the figures are conservative).  The first (full) step and the cache-aware steps
        # are accounted separately: the cache-aware step is the hot path proper.
        profs = {}

        def split(t):
            if t == 0:
                profs["full"] = m.profile_end()
                m.profile_begin()

        m.profile_begin()
        gen.run(hidden0, after_step=split)
        profs["cache_aware"] = m.profile_end()
        kernels = kernel_table(profs["cache_aware"], algorithmic_work(cfg, sched[1:]), peaks, "hbm")
        line["kernels"] = kernels
        line["kernels_scope"] = "the %d cache-aware steps of one generation" % (cfg.T - 1)
        line["full_step_kernels"] = kernel_table(profs["full"], algorithmic_work(cfg, sched[:1]), peaks, "tensor")
        dom = kernels[0]
        key = "gemm" if dom["bound"] == "tensor" else dom["kernel"]
        line["roofline"] = {"kernel": dom["kernel"], "bound": dom["bound"], "achieved": dom["achieved"], "peak": dom["peak"],
                            "unit": dom["unit"], "frac": dom["frac"], "traffic": load_ncu_traffic().get(key),
                            "peak_source": "%s (%s)" % (peak_kind, "sustained bf16 GEMM" if dom["bound"] == "tensor" else "device copy"),
                            "timing": "CUDA events in front of every launch, cache-aware steps of one generation of the timed workload"}

        # ---- cost of each kernel class inside the REAL chain (launch overlap on, no events between
        # kernels): the same generation with every launch of that class issued twice, minus the timed
        # generation.  (Leaving a class out instead would also raise the clocks of everything else on a
        # power-capped GPU; it is used only for the small remainder.)
        if n_dec is None:
            in_chain = {}
            names = ("gather_layernorm", "gemm_qkv", "attention", "gemm_out_proj", "gemm_fc1_gelu", "gemm_fc2")
            ms_ref = timed(lambda: gen.run(hidden0), 2)
            for cls in names:
                m.debug_repeat_classes([cls])
                gen.run(hidden0)
                in_chain[cls] = timed(lambda: gen.run(hidden0), 2) - ms_ref
            m.debug_repeat_classes(())
            m.debug_skip_classes(names)
            gen.run(hidden0)
            ms_rest = timed(lambda: gen.run(hidden0), 2)
            m.debug_skip_classes(())
            gen.run(hidden0)                                   # leaves the buffers of a real generation behind
            m.clear_device_status()
            w_all = algorithmic_work(cfg, sched)
            tot = sum(w_all["gemm_split"].values())
            rows_ic = []
            for cls in names:
                ms = in_chain[cls]
                if cls.startswith("gemm"):
                    amount, peak, unit = w_all["gemm_flops"] * w_all["gemm_split"][cls] / tot / 1e12, peaks["bf16_tflops_sustained"], "TFLOP/s"
                elif cls == "attention":
                    amount, peak, unit = w_all["attention_bytes"] / 1e9, peaks["hbm_gbs"], "GB/s"
                else:
                    amount, peak, unit = w_all["gather_layernorm_bytes"] / 1e9, peaks["hbm_gbs"], "GB/s"
                ach = amount / (ms * 1e-3) if ms > 0 else None
                rows_ic.append({"kernel": cls, "ms": ms, "share": ms / ms_ref, "achieved": ach, "unit": unit, "peak": peak,
                                "frac": None if ach is None else ach / peak})
            gemm_ms = sum(in_chain[c] for c in names if c.startswith("gemm"))
            line["kernels_in_chain"] = {
                "method": "the whole generation (all %d steps, full step included) with every launch of the class issued "
                          "twice, minus the generation as timed; launch overlap stays on; everything_else = the generation "
                          "with all six classes left out" % cfg.T,
                "ms_per_step": ms_ref, "rows": rows_ic, "everything_else_ms": ms_rest,
                "sum_ms": sum(in_chain.values()) + ms_rest,
                "gemm_all": {"ms": gemm_ms, "achieved": w_all["gemm_flops"] / 1e12 / (gemm_ms * 1e-3), "unit": "TFLOP/s",
                             "frac": w_all["gemm_flops"] / 1e12 / (gemm_ms * 1e-3) / peaks["bf16_tflops_sustained"]}}
            if dom["bound"] == "tensor":
                line["roofline"]["frac_in_chain"] = line["kernels_in_chain"]["gemm_all"]["frac"]
                line["roofline"]["achieved_in_chain"] = line["kernels_in_chain"]["gemm_all"]["achieved"]

        # ---- per-step latency: events between the steps of one more generation
        if n_dec is None:
            evs = [torch.cuda.Event(enable_timing=True) for _ in range(cfg.T + 1)]
            evs[0].record()
            gen.run(hidden0, after_step=lambda t: evs[t + 1].record())
            torch.cuda.synchronize()
            lat = [evs[t].elapsed_time(evs[t + 1]) for t in range(cfg.T)]
            line["step_latency_ms"] = {"full_step_t0": lat[0], "cache_aware_median": float(np.median(lat[1:])),
                                       "cache_aware_min": float(np.min(lat[1:])), "cache_aware_max": float(np.max(lat[1:])),
                                       "note": "includes the overwrite of the generated rows after each step"}

        # ---- each kernel on its own at the median cache-aware shape (no dependency gaps)
        n_mid = int(np.median([s_[1] for s_ in sched[1:]]))
        line["kernels_isolated"] = {"n_active": n_mid, "rows": isolated_kernels(m, cfg, peaks, n_mid, args.operand)}

        # ---- this build's own full-recompute path (full step at every decoding step)
        gen.run(hidden0, mode="full")
        ms_full = timed(lambda: gen.run(hidden0, mode="full"), 1)
        line["full_recompute"] = {"value": world * n_images / (ms_full * 1e-3), "unit": "images/s", "ms_per_step": ms_full,
                                  "speedup_cache_aware": ms_full / ms_gen}

        # ---- the paper's own schedule (Section 4.3): blocks up to the scoring block full in every step,
        # selection inside the step, fixed active budget of 64 rows, full refresh every 3rd step
        if cfg.score_layer < cfg.L - 1:
            gen.run_in_step(hidden0)
            ms_paper = timed(lambda: gen.run_in_step(hidden0), 2)
            line["paper_schedule"] = {"value": world * n_images / (ms_paper * 1e-3), "unit": "images/s",
                                      "ms_per_step": ms_paper,
                                      "speedup_vs_full_recompute": ms_full / ms_paper, "active_budget": 64,
                                      "full_refresh_period": 3, "score_layer": cfg.score_layer,
                                      "paper_reports": "1.68x end to end for MAR-L on one H100 (Table 1), sampler included"}

        # ---- the two-stage model (Eq. 1, Eq. 2): encoder blocks on the known tokens only, recomputed in
        # every step; decoder under the same schedule.  This is the shape the paper's own numbers are for.
        if 1 <= cfg.E < cfg.L and cfg.score_layer < cfg.L - 1:
            from paper_2506_12035_b200.binding import upload_mar_weights
            m.set_mar_weights(upload_mar_weights(synth.make_mar_weights(cfg), cfg.dtype, operand=args.operand))
            known = synth.known_token_sets(cfg, sets)
            gen.run_mar(hidden0, known)
            ms_ts = timed(lambda: gen.run_mar(hidden0, known), 2)
            gen.run_mar(hidden0, known, mode="full")
            ms_ts_full = timed(lambda: gen.run_mar(hidden0, known, mode="full"), 2)
            line["two_stage"] = {"value": world * n_images / (ms_ts * 1e-3), "unit": "images/s", "ms_per_step": ms_ts,
                                 "full_recompute_ms_per_step": ms_ts_full,
                                 "speedup_vs_full_recompute": ms_ts_full / ms_ts, "active_budget": 64,
                                 "full_refresh_period": 3, "score_layer": cfg.score_layer,
                                 "encoder": "known tokens only, every step; decoder cache-aware",
                                 "paper_reports": "1.68x end to end for MAR-L on one H100 (Table 1), sampler included"}
            assert m.device_status() == 0

        # ---- end to end through marche_step_host: pinned host buffers, copies inside the timed region
        gen.alloc_host_buffers(hidden0_np, rows_np, sets)
        for _ in range(2):
            h2d, d2h = gen.run_host()
        e2e_fn, e2e_launch = (lambda: gen.run_host()), "stream launches"
        if graph is not None:
            # the same calls recorded once: the copies from / to the pinned host buffers become graph nodes
            try:
                side = torch.cuda.Stream()
                g_e2e = torch.cuda.CUDAGraph()
                with torch.cuda.stream(side):
                    with torch.cuda.graph(g_e2e, stream=side):
                        gen.run_host()
                g_e2e.replay()
                torch.cuda.synchronize()
                e2e_fn, e2e_launch = (lambda: g_e2e.replay()), "one CUDA graph per generation, copies as graph nodes"
            except Exception as exc:
                e2e_launch = "stream launches (graph capture failed: %s)" % str(exc)[:120]
        ms_e2e = timed(e2e_fn, args.steps)
        line["e2e"] = {"value": world * n_images / (ms_e2e * 1e-3), "unit": "images/s", "h2d_bytes_per_step": int(h2d),
                       "d2h_bytes_per_step": int(d2h), "ms_per_step": ms_e2e, "launch": e2e_launch,
                       "api": "marche_step_host: per step, inputs from pinned host memory, results back to it"}
        assert m.device_status() == 0

        # ---- CPU oracle on a bounded sample (rank 0, N = 1 only)
        if world == 1 and not args.no_cpu_baseline:
            ips, _, info = oracle_sample(cfg, ratio)
            line["cpu_baseline"] = dict(info, value=ips, unit="images/s")
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def isolated_kernels(m, cfg, peaks, n_active, operand="f16"):
    """Each hot-path kernel timed on its own at one mid-run shape (n_active rows per sample):
    back-to-back launches through the single-kernel C calls (replayed from a CUDA graph), CUDA events around the batch, buffers
    rotated so that streamed operands come from HBM.  Unlike the per-class table of the generation,
    these figures contain no dependency gaps: they are the kernels' own roofline fractions."""
    import torch
    B, S, D, F, H = cfg.B, cfg.S, cfg.D, cfg.F, cfg.H
    M = B * n_active
    dev = "cuda"
    act = (torch.float16 if operand == "f16" else torch.bfloat16) if cfg.dtype == "bf16" else torch.float32
    typ = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    eb = 2 if cfg.dtype == "bf16" else 4
    rot = 3
    xs = [torch.randn(M, D, device=dev) for _ in range(rot)]
    us = [torch.empty(M, D, device=dev, dtype=act) for _ in range(rot)]
    qkvs = [torch.randn(M, 3 * D, device=dev).to(typ) for _ in range(rot)]
    caches = [torch.randn(2, B, S, D, device=dev).to(typ) for _ in range(rot)]
    o = torch.empty(M, D, device=dev, dtype=act)
    g = torch.empty(M, F, device=dev, dtype=act)
    idx = torch.stack([torch.randperm(S, device=dev)[:n_active] for _ in range(B)]).to(torch.int32).contiguous()
    w0 = m.weights[0]
    partial = torch.rand(B, H, S, device=dev)
    scores = torch.rand(B, S, device=dev)
    mask = torch.empty(B * S, dtype=torch.uint8, device=dev)
    k = int(np.floor(cfg.ratio * S + 0.5))
    refresh = torch.empty(B, max(k, 1), dtype=torch.int32, device=dev)
    new = idx[:, :4].contiguous()

    def timed_us(fn, reps=24):
        # the launches are recorded into a CUDA graph and replayed, so that the host's per-call cost
        # (several microseconds through the Python binding) does not bound the small kernels
        for i in range(3):
            fn(i)
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                for i in range(reps):
                    fn(i)
        graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        graph.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps * 1e3

    rows = []

    def add(name, bound, amount, us):
        unit = "TFLOP/s" if bound == "tensor" else "GB/s"
        # a kernel timed alone in a short burst runs at boost clocks: the burst GEMM peak is its denominator
        # (the generation as a whole runs under the power cap and is compared with the sustained peak)
        peak = peaks["bf16_tflops"] if bound == "tensor" else peaks["hbm_gbs"]
        ach = amount / (us * 1e-6) / (1e12 if bound == "tensor" else 1e9)
        rows.append({"kernel": name, "bound": bound, "us": us, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak})

    add("gather_layernorm (M x D)", "hbm", M * D * (4 + eb),
        timed_us(lambda i: m.gather_layernorm(xs[i % rot].view(B, n_active, D), None, n_active, w0["ln2_g"], w0["ln2_b"], None, us[i % rot])))
    add("scatter_kv", "hbm", 4.0 * M * D * eb,
        timed_us(lambda i: m.scatter_kv(qkvs[i % rot][:, D:], qkvs[i % rot][:, 2 * D:], 3 * D, idx, n_active, caches[i % rot])))
    add("attention (plain)", "hbm", 2.0 * B * S * D * eb + 2.0 * M * D * eb,
        timed_us(lambda i: m.attention(qkvs[i % rot], 3 * D, n_active, caches[i % rot], None, None, o)))
    for name, a_in, wname, bname, epi, out, N, K in (
            ("gemm qkv", us[0], "w_qkv", "b_qkv", 0, qkvs[0], 3 * D, D), ("gemm out-proj (+residual)", o, "w_o", "b_o", 1, xs[0], D, D),
            ("gemm fc1 (+GELU)", us[0], "w_fc1", "b_fc1", 2, g, F, D), ("gemm fc2 (+residual)", g, "w_fc2", "b_fc2", 1, xs[0], D, F)):
        add("%s %dx%dx%d" % (name, M, N, K), "tensor", 2.0 * M * N * K,
            timed_us(lambda i: m.linear(a_in, w0[wname], w0[bname], epi, out)))
    add("topk (select_refresh, k=%d)" % k, "hbm", B * S * 5 + B * k * 4,
        timed_us(lambda i: m.select_refresh(scores, new, None, k, refresh, mask)))
    return rows


def run_microbench(args):
    """Appendix B on B200: attention over a fresh segment of n rows and a cached segment, (i) write
    the fresh K/V into the cache and run the one-segment kernel over everything (the in-place
    equivalent of "concatenate, then standard kernel"), (ii) the two-segment kernel that reads the
    fresh segment in place, merges by online softmax and writes the cache back afterwards.
    MAR-L layer shape (B 128, 16 heads of 64).  One JSON line per length pair."""
    import torch
    from paper_2506_12035_b200.binding import Marche, upload_weights
    base = synth.CONFIGS["mar_l"].replace(L=1, E=0)
    blocks = synth.make_weights(base)
    w = upload_weights(blocks, "bf16")
    for fresh, cached in ((32, 256), (16, 256), (64, 256), (128, 256), (41, 279), (32, 1024), (128, 960)):
        cfg = base.replace(S=fresh + cached)
        m = Marche.from_config(cfg, w)
        B, S, D, H = cfg.B, cfg.S, cfg.D, cfg.H
        caches = [torch.randn(2, B, S, D, device="cuda").to(torch.bfloat16) for _ in range(3)]   # rotate: > L2
        qkv = torch.randn(B * fresh, 3 * D, device="cuda").to(torch.bfloat16)
        o = torch.zeros(B * fresh, D, device="cuda", dtype=torch.float16)
        idx = torch.stack([torch.randperm(S, device="cuda")[:fresh] for _ in range(B)]).to(torch.int32).contiguous()

        def one(i):
            m.scatter_kv(qkv[:, D:], qkv[:, 2 * D:], 3 * D, idx, fresh, caches[i % 3])
            m.attention(qkv, 3 * D, fresh, caches[i % 3], None, None, o)

        def two(i):
            m.attention_two_segment(qkv, 3 * D, fresh, idx, caches[i % 3], None, None, o)

        res = {}
        for name, fn in (("scatter_then_attend_us", one), ("two_segment_us", two)):
            for i in range(3):
                fn(i)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(24):
                fn(i)
            e1.record()
            torch.cuda.synchronize()
            res[name] = e0.elapsed_time(e1) / 24 * 1e3
        assert m.device_status() == 0
        res.update({"microbench": "attention, fresh + cached segments (Appendix B)", "fresh": fresh, "cached": cached,
                    "batch": B, "heads": H, "head_dim": cfg.dh,
                    "latency_change": res["two_segment_us"] / res["scatter_then_attend_us"] - 1.0,
                    "paper_reports": "-19.2 % at (32, 256) on its hardware, -16.2 .. -27.3 % overall"})
        print(json.dumps(res), flush=True)

    # ---- K4 at scale: the per-step call (B 128) is latency-bound and cannot show a bandwidth figure, so
    # the same two kernels (candidate flags, radix select) are also run on many samples.
    peaks, _ = load_peaks()
    for Bk, Sk, k in ((128, 320, 32), (16384, 320, 32), (16384, 1088, 109)):
        small = synth.CONFIGS["tiny"].replace(L=1, E=0, D=128, H=2, F=128, S=Sk, B=Bk, dtype="bf16")
        m = Marche.from_config(small, upload_weights(synth.make_weights(small), "bf16"))
        scores = torch.rand(Bk, Sk, device="cuda")
        new = torch.stack([torch.randperm(Sk, device="cuda")[:4] for _ in range(min(Bk, 256))]).to(torch.int32)
        new = new.repeat((Bk + new.shape[0] - 1) // new.shape[0], 1)[:Bk].contiguous()
        out = torch.empty(Bk, k, dtype=torch.int32, device="cuda")
        mask = torch.empty(Bk * Sk, dtype=torch.uint8, device="cuda")
        for _ in range(3):
            m.select_refresh(scores, new, None, k, out, mask)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(10):
            m.select_refresh(scores, new, None, k, out, mask)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / 10 * 1e3
        nbytes = Bk * Sk * 5 + Bk * k * 4 + Bk * Sk          # scores + mask read, indices written, mask written
        print(json.dumps({"microbench": "top-k refresh selection (flags + radix select)", "batch": Bk, "seq_len": Sk, "k": k,
                          "us": us, "GB/s": nbytes / us * 1e-3, "frac_of_hbm": nbytes / us * 1e-3 / peaks["hbm_gbs"]}), flush=True)


def spawn_replicas(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: starts one replica process per GPU with the
    environment a launcher would have set (rank 0's JSON line goes to this process's stdout)."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env))
    return max(p.wait() for p in procs)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="mar_l", choices=list(synth.CONFIGS))
    ap.add_argument("--ratio", type=float, default=0.10)
    ap.add_argument("--blocks", type=int, default=0, help="override the depth (profiling captures only)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch (profiling captures only)")
    ap.add_argument("--tsteps", type=int, default=0, help="override the decoding steps (profiling captures only)")
    ap.add_argument("--decode-steps", type=int, default=0,
                    help="stop each generation after this many decoding steps (profiling captures only)")
    ap.add_argument("--no-extras", action="store_true", help="only the timed region (for ncu launch lists)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--stream-launch", action="store_true",
                    help="time the stream-launched generation instead of its CUDA-graph replay")
    ap.add_argument("--microbench", action="store_true",
                    help="Appendix-B style attention micro-benchmark instead of the generation benchmark")
    ap.add_argument("--operand", default="f16", choices=["f16", "bf16"],
                    help="16-bit configs: element type of the projections' operands (f16 meets the 3e-2 bound at full depth)")
    ap.add_argument("--write-traffic", default="", help="ncu raw csv -> profiles/ncu_dram_traffic.txt, then exit")
    args = ap.parse_args()
    if args.write_traffic:
        write_ncu_traffic(args.write_traffic)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.microbench:
        sys.exit(spawn_replicas(args.gpus))
    cfg = synth.CONFIGS[args.config]
    if args.blocks:
        cfg = cfg.replace(L=args.blocks, E=min(cfg.E, max(0, args.blocks - 2)))
    if args.batch:
        cfg = cfg.replace(B=args.batch)
    if args.tsteps:
        cfg = cfg.replace(T=args.tsteps)
    if args.microbench:
        run_microbench(args)
    elif args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
