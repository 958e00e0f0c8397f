#!/usr/bin/env python
"""Benchmark of the AAAC per-layer quantisation path on B200.

One step = the whole hot path over one batch of synthetic layers: for each layer activation
statistics, scales, quantile initialisation, R fit rounds, the final pack pass and a
dequantisation.  The workload is the Llama-3-8B-shaped configuration (q_proj 4096x4096,
gate_proj 14336x4096, down_proj 4096x14336; NVFP4, group 16, 4096 calibration tokens, 20
rounds) on seeded synthetic data.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints one JSON line (rank 0).  With N > 1 (under torchrun) every rank quantises its own
batch of layers (independent problems, no data-path collective): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "aaac_fit_throughput"
UNIT = "Gweights/s per k-means round"
ROUNDS = 20
TOKENS = 4096
LAYERS = ["q_proj", "gate_proj", "down_proj"]
BYTES_PER_WEIGHT = 2.0 + 1.0 / 16.0          # NVFP4 fit round: BF16 weight + E4M3 scale per 16
REPEATS = 5                                  # the K-step timed loop is repeated; the median is reported
# algorithmic bytes per weight of the other stages of a step (NVFP4 g16; X is counted per element)
STAGE_BYTES = {
    "act_stats": None,                       # 2 B per element of X read, 4 B per input channel written
    "scales": 2 * 2.0 + 1.0 / 16.0,          # layer absmax pass + group pass over W, E4M3 scales written
    "quantile_init": 3 * 2.0,                # a three-pass exact selection over W (the path makes two passes)
    "pack": BYTES_PER_WEIGHT + 0.5 + 1.0 / 16.0,   # W + scales read, codes and scale sign bits written
    "dequant": 0.5 + 1.0 / 16.0 + 2.0,       # codes + scales read, BF16 weights written
}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


TRAFFIC_FILE = os.path.join("profiles", "fit_batch_cfg2_full_step.md")


def measured_traffic_per_weight():
    """DRAM bytes per weight and round of the fit-rounds kernel, from the line
    `dram_bytes_per_weight_round = X` of the committed ncu summary (None if absent).  It is a
    constant taken from one earlier capture on one layer, not a measurement of this run."""
    p = os.path.join(ROOT, TRAFFIC_FILE)
    try:
        for line in open(p):
            if line.strip().startswith("dram_bytes_per_weight_round"):
                return float(line.split("=")[1].split()[0])
    except Exception:
        pass
    return None


class ClockSampler:
    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-lms", "20",
                                       "-i", str(index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def count(self) -> int:
        """Samples written so far."""
        try:
            self.f.flush()
            with open(self.f.name) as g:
                return sum(1 for line in g if line.count(",") >= 8)
        except OSError:
            return 0

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                mx.append(float(c[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if sm:
            busy = [s for s in sm if s > 0]
            out = {"sm_mhz": float(np.median(busy)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                   "samples": len(sm)}
        return out


def make_layers(seed, names=None):
    from paper_2605_08692_b200 import synth
    return [synth.config2_layer(w, seed=seed, tokens=TOKENS) for w in (names or LAYERS)]


def cpu_baseline_sample(layers, rounds=ROUNDS, rows=None):
    """The oracle, as it stands, on a bounded sample of the workload: the fit rounds (scales and
    quantile init excluded) of the given layers, optionally only their first `rows` rows, on all
    host cores."""
    import oracle
    total_w, dt, names = 0, 0.0, []
    for c in layers:
        W = np.ascontiguousarray(c["W"][:rows]) if rows else c["W"]
        I = oracle.act_stats(c["X"][:256])
        s, ts = oracle.scales(W, c["mode"], c["group"])
        wt = oracle.normalise(W, c["mode"], c["group"], s, ts)
        T = oracle.init_quantile(wt)
        t0 = time.perf_counter()
        for _ in range(rounds):
            T, _ = oracle.fit_round(wt, I, c["group"], T)
        dt += time.perf_counter() - t0
        total_w += W.size
        names.append(f"{c['name'].split('/')[-1]} {W.shape[0]}x{W.shape[1]}")
    return total_w * rounds / dt / 1e9, oracle.max_threads(), f"{rounds} fit rounds of " + ", ".join(names), dt


def run_reference(args, rank):
    """Reference arm = the CPU oracle, as it stands, on the same workload as the library's arm (the
    fit rounds of the three cfg2 layers).  A step is the whole workload when the requested number of
    steps fits into a few minutes at the oracle's rate; otherwise the first rows of every layer, as
    many as keep the run near two minutes (the sample is stated in the line)."""
    if rank != 0:
        return
    from paper_2605_08692_b200 import synth
    total_steps = args.warmup + args.steps
    full_step_s = 9.0                                    # the whole workload on about 16 host cores
    frac = min(1.0, args.ref_seconds / (full_step_s * max(total_steps, 1)))
    # generate only the rows that are used (rows are generated independently of N), and the 256
    # tokens the importance of the sample is taken from
    layers = [synth.config2_layer(w, seed=0, tokens=256,
                                  rows=None if frac >= 1.0 else max(64, int(synth.LLAMA8B_LINEARS[w][0] * frac) // 64 * 64))
              for w in LAYERS]
    vals, sample, cores = [], "", 0
    for i in range(total_steps):
        tw, dt_sum, names = 0, 0.0, []
        for c in layers:
            rows = None if frac >= 1.0 else max(64, int(c["W"].shape[0] * frac) // 64 * 64)
            v, cores, smp, dt = cpu_baseline_sample([c], rounds=ROUNDS, rows=rows)
            tw += (c["W"].shape[0] if rows is None else rows) * c["W"].shape[1]
            dt_sum += dt
            names.append(smp.split(" of ", 1)[1])
        sample = f"{ROUNDS} fit rounds of " + ", ".join(names) + (" (whole workload)" if frac >= 1.0 else " (first rows of every layer)")
        if i >= args.warmup:
            vals.append((tw * ROUNDS / dt_sum / 1e9, dt_sum))
    value = float(np.median([v for v, _ in vals]))
    ms = float(np.median([d for _, d in vals]) * 1e3)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": CFG2_WORKLOAD, "weights_per_step": int(sum(c["W"].size for c in layers)), "rounds": ROUNDS,
                       "note": "the CPU oracle times the fit rounds only (scales, quantile start and pack excluded)"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


CFG2_WORKLOAD = ("cfg2: Llama-3-8B-shaped q_proj 4096x4096, gate_proj 14336x4096, down_proj 4096x14336; NVFP4 g16 E4M3 "
                 "scales; X 4096 tokens; quantile init; 20 rounds; step = act_stats + scales + init + 20 fit rounds + "
                 "pack + dequant of the three layers (one aaac_quantize_layers call)")

STACKS = {
    # name: (decoder layers, hidden, kv width, intermediate, mode, tokens, rounds)
    "stack8b": (32, 4096, 1024, 14336, 0, 16384, 20),     # Llama-3-8B-shaped, INT4 g128
    "stack7b": (28, 3584, 512, 18944, 1, 16384, 20),      # Qwen2.5-7B-shaped, NVFP4 g16
}


def run_stack(args, which, emit=True):
    """Wall time of a whole decoder stack of random weights: per decoder layer four activation
    matrices (attention input shared by q/k/v, o input, MLP input shared by gate/up, down input) and
    seven linears, each through act_stats (once per distinct input), scales, quantile init, the fit
    rounds and the pack pass.  The layers of a stack are i.i.d. synthetic, so one decoder layer's
    tensors are generated on the device (seeded torch generator, outside the timed region) and the
    per-layer path is run once per decoder layer on them; every linear re-reads its W from HBM
    (one decoder layer touches > 1 GB, far more than the L2)."""
    import torch
    from paper_2605_08692_b200 import binding, build
    build.build()
    L, H, KV, FF, mode, tokens, rounds = STACKS[which]
    n_inner = 1
    if args.budget:                      # e.g. 3,10: the paper's default (n_outer, n_inner)
        rounds, n_inner = (int(v) for v in args.budget.split(","))
    g = 128 if mode == 0 else 16
    sel = args.sel_group or None          # None: S = g, selection bit in the scale's sign
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)

    def weights(n, k, t5=False):
        w = torch.randn(n, k, device=dev, generator=gen)
        if t5:
            chi = sum(torch.randn(n, k, device=dev, generator=gen) ** 2 for _ in range(5)) / 5.0
            w = w / chi.sqrt()
        return (w * 0.02).to(torch.bfloat16)

    def acts(k):
        c = torch.exp(torch.randn(k, device=dev, generator=gen))
        c[torch.randperm(k, device=dev, generator=gen)[: max(1, k // 200)]] *= 30.0
        return (torch.randn(tokens, k, device=dev, generator=gen) * c).to(torch.bfloat16)

    t5 = which == "stack7b"
    X = {"attn": acts(H), "o": acts(H), "mlp": acts(H), "down": acts(FF)}
    lin = [("q", H, H, "attn"), ("k", KV, H, "attn"), ("v", KV, H, "attn"), ("o", H, H, "o"),
           ("gate", FF, H, "mlp"), ("up", FF, H, "mlp"), ("down", H, FF, "down")]
    Ws = {n: weights(N, K, t5) for n, N, K, _ in lin}
    out = {}
    for n, N, K, _ in lin:
        out[n] = dict(T01=torch.zeros(2, 16, dtype=torch.float32, device=dev),
                      Tb=torch.empty(2, 16, dtype=torch.uint16, device=dev),
                      scales=torch.empty(N, K // g, dtype=torch.uint16 if mode == 0 else torch.uint8, device=dev),
                      ts=torch.ones(1, dtype=torch.float32, device=dev),
                      codes=torch.empty(N, K // 2, dtype=torch.uint8, device=dev),
                      err=torch.zeros(2, dtype=torch.float64, device=dev),
                      bits=torch.empty(N, K // (8 * sel), dtype=torch.uint8, device=dev) if sel and sel != g else None,
                      ws=binding.alloc_workspace(mode, N, K, tokens, dev))
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    # the seven linears of a decoder layer are independent: one aaac_quantize_layers call (importances -- once per
    # distinct input: q, k, v share theirs, gate and up too --, scales, start, rounds in one launch, pack)
    descs = [dict(W=Ws[n], X=X[xin], T01=out[n]["T01"], scales=out[n]["scales"], tensor_scale=out[n]["ts"], ws=out[n]["ws"],
                  T01_bf16=out[n]["Tb"], codes=out[n]["codes"], err_out=out[n]["err"], sigma_bits=out[n]["bits"])
             for n, N, K, xin in lin]

    def decoder_layer():
        binding.quantize_layers(descs, mode, n_outer=rounds, n_inner=n_inner, init=binding.INIT_QUANTILE, dev_status=status,
                                sel_group=sel)

    for _ in range(2):
        decoder_layer()
    torch.cuda.synchronize()
    # kernels of one decoder layer: act_stats 2 per input; per linear absmax (NVFP4) + scales, 6 of the
    # quantile start, the fit launches, export, pack + its export
    n0 = binding.launch_count()
    decoder_layer()
    launches_per_layer = binding.launch_count() - n0
    sampler = ClockSampler(0)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(L):
        decoder_layer()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if int(status.item()) != 0:
        raise SystemExit("device status is set")
    wall = e0.elapsed_time(e1) * 1e-3
    wl = sum(N * K for _, N, K, _ in lin)
    line = {"metric": "aaac_stack_wall_s", "value": wall, "unit": "s", "n_gpus": 1, "higher_is_better": False,
            "dtype": "f32", "data": "synthetic (device-generated, one decoder layer's tensors reused for every layer)",
            "config": {"workload": f"{which}: {L} decoder layers x 7 linears (hidden {H}, kv {KV}, intermediate {FF}), "
                                   f"{'INT4 g128' if mode == 0 else 'NVFP4 g16'} S{sel or g}, {tokens} tokens per input, quantile init, "
                                   f"n_outer {rounds}, n_inner {n_inner}; act_stats + scales + init + rounds + pack (the seven linears of a "
                                   f"decoder layer in one aaac_quantize_layers call)",
                       "linears": 7 * L, "weights": wl * L, "rounds": rounds, "n_inner": n_inner},
            "gweights_per_s_per_round": wl * L * rounds * n_inner / wall / 1e9, "clocks": clocks,
            "gpu_launches": launches_per_layer * L}
    del X, Ws, out
    torch.cuda.empty_cache()
    if emit:
        print(json.dumps(line), flush=True)
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--ref-seconds", type=float, default=120.0,
                    help="reference arm: CPU seconds the whole run should take (bounds the sample per step)")
    ap.add_argument("--with-prescale", action="store_true",
                    help="profiling runs: also scale every layer's input channels (aaac_prescale_columns, unit "
                         "multipliers) at the start of a step, so that the kernel shows up in a capture")
    ap.add_argument("--no-stacks", action="store_true",
                    help="leave the decoder-stack wall times out of the line (profiling runs)")
    ap.add_argument("--layers", default=",".join(LAYERS),
                    help="subset of the workload's layers (profiling a small case); the default is the full workload")
    ap.add_argument("--workload", default="cfg2", choices=["cfg2"] + sorted(STACKS),
                    help="cfg2 (default): the benchmark contract; stack8b / stack7b: wall time of a whole decoder stack")
    ap.add_argument("--budget", default="",
                    help="stack workloads only: n_outer,n_inner (default: the workload's rounds with n_inner = 1)")
    ap.add_argument("--sel-group", type=int, default=0,
                    help="stack workloads only: selection group size S (default: the scale group; 16 with stack8b "
                         "is the paper's INT4 g128 S16 variant)")
    args = ap.parse_args()
    if args.workload != "cfg2":
        if int(os.environ.get("RANK", "0")) == 0:
            run_stack(args, args.workload)
        return

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        # no launcher set the ranks up: start one process per GPU ourselves
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2605_08692_b200 import binding, build, sharding
    build.build()
    binding.lib()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    warmup = max(args.warmup, 3)
    names = [n for n in args.layers.split(",") if n]
    layers = make_layers(seed=sharding.seed_for_rank(0, rank), names=names)
    mode = layers[0]["mode"]

    def to_dev(a):
        return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)

    Wd = [to_dev(c["W"]) for c in layers]
    Xd = [to_dev(c["X"]) for c in layers]
    shapes = [tuple(c["W"].shape) for c in layers]
    weights_per_step = sum(n * k for n, k in shapes)
    # device outputs and scratch, allocated once
    outs = []
    for (N, K) in shapes:
        outs.append(dict(
            I=torch.empty(K, dtype=torch.float32, device=dev),
            T01=torch.zeros(2, 16, dtype=torch.float32, device=dev),
            Tb=torch.empty(2, 16, dtype=torch.uint16, device=dev),
            scales=torch.empty(N, K // 16, dtype=torch.uint8, device=dev),
            ts=torch.ones(1, dtype=torch.float32, device=dev),
            codes=torch.empty(N, K // 2, dtype=torch.uint8, device=dev),
            err=torch.zeros(2, dtype=torch.float64, device=dev),
            What=torch.empty(N, K, dtype=torch.bfloat16, device=dev),
            ws=binding.alloc_workspace(mode, N, K, TOKENS, dev)))
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    descs = [dict(W=W, X=X, T01=o["T01"], scales=o["scales"], tensor_scale=o["ts"], ws=o["ws"], T01_bf16=o["Tb"],
                  codes=o["codes"], err_out=o["err"], What=o["What"]) for W, X, o in zip(Wd, Xd, outs)]
    descs_I = [dict(d, X=None, I=o["I"]) for d, o in zip(descs, outs)]
    ones = {K: torch.ones(K, dtype=torch.float32, device=dev) for _, K in shapes} if args.with_prescale else {}

    def step():
        # the layers of a step are independent problems: one aaac_quantize_layers call takes them through the
        # whole path (importances from X, scales, start tables, the 20 rounds of all of them in one launch,
        # pack, reconstruction)
        if args.with_prescale:
            for X, W, o in zip(Xd, Wd, outs):
                binding.act_stats(X, o["I"], o["ws"], dev_status=status)
                binding.prescale_columns(W, ones[W.shape[1]], o["What"], o["I"], o["I"], dev_status=status)
            binding.quantize_layers(descs_I, mode, n_outer=ROUNDS, init=binding.INIT_QUANTILE, dev_status=status)
            return
        binding.quantize_layers(descs, mode, n_outer=ROUNDS, init=binding.INIT_QUANTILE, dev_status=status)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # the clock sampler starts before the warm-up steps: the query tool needs longer to start than a
    # short timed region lasts
    sampler = ClockSampler(local_rank) if rank == 0 else None
    for _ in range(warmup):
        step()
    barrier()
    # EXACTLY --steps steps between a barrier + synchronise on both sides, device-timed; that
    # measurement is repeated and the median repeat is the one reported (a few-millisecond step
    # makes a single short region jumpy)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = []
    for _ in range(REPEATS):
        binding.timing_begin(args.steps)
        n0 = binding.launch_count()
        barrier()
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        barrier()
        launches = binding.launch_count() - n0
        ms_rep = sharding.max_over_ranks(e0.elapsed_time(e1), dev)
        reps.append((ms_rep, binding.timing_end(args.steps), launches))   # one entry per fit launch (all rounds of the step's layers)
    reps.sort(key=lambda r: r[0])
    ms_total, round_ms, launches = reps[len(reps) // 2]
    clocks = None
    if sampler:
        # a timed region of a few milliseconds can end before the first sample: keep the same load
        # running, untimed, until a few samples exist (at most two seconds)
        extra, t_end = 0, time.time() + 2.0
        while sampler.count() < 5 and time.time() < t_end:
            step()
            torch.cuda.synchronize()
            extra += 1
        clocks = sampler.stop()
        clocks["window"] = f"warm-up and timed steps, plus {extra} untimed steps of the same load"
    if int(status.item()) != 0:
        raise SystemExit("device status reports non-finite input")
    ms_step = ms_total / args.steps
    value = sharding.job_throughput(weights_per_step, ROUNDS, ms_step, world)

    # roofline of the dominant kernel: algorithmic bytes of every timed fit-round launch / its device time
    per_launch_w = [weights_per_step * ROUNDS] * args.steps
    bytes_alg = sum(per_launch_w[:len(round_ms)]) * BYTES_PER_WEIGHT
    fit_ms = float(sum(round_ms))
    achieved = bytes_alg / (fit_ms * 1e-3) / 1e9 if fit_ms > 0 else 0.0
    peak, peak_kind = peaks()
    tpw = measured_traffic_per_weight()
    roofline = {"kernel": "fit_batch_kernel (one launch = the 20 k-means rounds of the step's layers, each layer on its share "
                          "of the blocks)" if len(layers) > 1 else "fit_rounds_kernel (one launch = the 20 k-means rounds of the layer)",
                "bound": "hbm",
                "binding_units": "by the ncu counters the kernel is held by the shared-memory data pipe and instruction "
                                 "issue, not by HBM; the HBM fraction is reported because it is the metric",
                "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "peak_source": f"of {peak_kind}",
                "traffic": None if tpw is None else tpw * float(np.mean(per_launch_w)),
                "traffic_source": None if tpw is None else f"{TRAFFIC_FILE} (a constant per weight and round from one "
                                                           "earlier ncu capture of this workload's launch; not measured "
                                                           "in this run)",
                "algorithmic_bytes_per_launch": float(np.mean(per_launch_w)) * BYTES_PER_WEIGHT,
                "avg_launch_ms": fit_ms / max(len(round_ms), 1),
                "fit_share_of_step": fit_ms / ms_total if ms_total > 0 else None,
                "gweights_per_s_kernel": sum(per_launch_w[:len(round_ms)]) / (fit_ms * 1e-3) / 1e9 if fit_ms else 0.0}

    # the other stages of a step, each bracketed by events inside steps of the same rotation (so a
    # layer's data has been evicted by the other layers' before it is used again); median over steps
    stage_names = ["act_stats", "scales+init+fit+export (layer by layer)", "pack", "dequant"]
    stage_ms = {k: [] for k in stage_names}
    split_ms = []                                               # scales + quantile init alone (fit with n_outer = 0)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(len(layers) * 5 * 2)]
    for rep in range(7):
        k = 0
        marks = []
        for W, X, o in zip(Wd, Xd, outs):
            ev[k].record(); binding.act_stats(X, o["I"], o["ws"], dev_status=status); ev[k + 1].record()
            ev[k + 2].record()
            binding.fit_layer(W, mode, I=o["I"], n_outer=ROUNDS, init=binding.INIT_QUANTILE, T01=o["T01"],
                              scales=o["scales"], tensor_scale=o["ts"], ws=o["ws"], dev_status=status)
            ev[k + 3].record()
            ev[k + 4].record()
            binding.pack(W, mode, I=o["I"], T01=o["T01"], T01_bf16=o["Tb"], scales=o["scales"], tensor_scale=o["ts"],
                         codes=o["codes"], ws=o["ws"], err_out=o["err"])
            ev[k + 5].record()
            ev[k + 6].record(); binding.dequant(o["codes"], o["scales"], o["ts"], o["Tb"], mode, o["What"]); ev[k + 7].record()
            marks.append(k)
            k += 10
        torch.cuda.synchronize()
        if rep >= 2:
            for j, name in enumerate(stage_names):
                stage_ms[name].append(sum(ev[m + 2 * j].elapsed_time(ev[m + 2 * j + 1]) for m in marks))
    for rep in range(7):
        k = 0
        for W, X, o in zip(Wd, Xd, outs):
            ev[k].record()
            binding.fit_layer(W, mode, I=o["I"], n_outer=0, init=binding.INIT_QUANTILE, T01=o["T01"],
                              scales=o["scales"], tensor_scale=o["ts"], ws=o["ws"], dev_status=status)
            ev[k + 1].record()
            binding.pack(W, mode, I=o["I"], T01=o["T01"], T01_bf16=o["Tb"], scales=o["scales"], tensor_scale=o["ts"],
                         codes=o["codes"], ws=o["ws"], err_out=o["err"])      # keeps the rotation's eviction pattern
            k += 10
        torch.cuda.synchronize()
        if rep >= 2:
            split_ms.append(sum(ev[m].elapsed_time(ev[m + 1]) for m in range(0, 10 * len(layers), 10)))
    x_elems = sum(int(x.numel()) for x in Xd)
    k_total = sum(K for _, K in shapes)
    med = {k: float(np.median(v)) for k, v in stage_ms.items()}
    scales_init_ms = float(np.median(split_ms))

    def stage(name, ms, nbytes, note=None):
        gbs = nbytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0
        d = {"stage": name, "ms_per_step": ms, "algorithmic_bytes_per_step": float(nbytes), "achieved": gbs, "unit": "GB/s",
             "peak": peak, "frac": gbs / peak}
        if note:
            d["note"] = note
        return d
    roofline_other = [
        stage("act_stats (act_sumsq_kernel + act_final_kernel)", med["act_stats"], 2.0 * x_elems + 4.0 * k_total),
        stage("scales + quantile start (absmax, scales, histogram, plan, collection, selection kernels)", scales_init_ms,
              (STAGE_BYTES["scales"] + STAGE_BYTES["quantile_init"]) * weights_per_step,
              "bytes: two passes for the NVFP4 scales plus a three-pass exact selection over W; the path itself reads W "
              "four times in this stage"),
        stage("pack (pack_kernel)", med["pack"], STAGE_BYTES["pack"] * weights_per_step),
        stage("dequant (dequant_kernel)", med["dequant"], STAGE_BYTES["dequant"] * weights_per_step),
    ]

    # end to end through the host-buffer entry point (pinned host memory in and out)
    e2e = None
    host = []
    try:
        for c, (N, K) in zip(layers, shapes):
            host.append(dict(
                W=torch.from_numpy(c["W"].view(np.int16)).pin_memory(), X=torch.from_numpy(c["X"].view(np.int16)).pin_memory(),
                T01=torch.empty(2, 16, dtype=torch.float32).pin_memory(), Tb=torch.empty(2, 16, dtype=torch.int16).pin_memory(),
                sc=torch.empty(N, K // 16, dtype=torch.uint8).pin_memory(), ts=torch.empty(1, dtype=torch.float32).pin_memory(),
                codes=torch.empty(N, K // 2, dtype=torch.uint8).pin_memory(), err=torch.empty(2, dtype=torch.float64).pin_memory(),
                status=torch.zeros(1, dtype=torch.int32).pin_memory(), stream=torch.cuda.Stream(device=dev),
                ws=torch.empty(binding.host_workspace_bytes(mode, N, K, TOKENS), dtype=torch.uint8, device=dev)))

        def host_step():
            # one stream and one workspace per layer: a layer's copies overlap the other layers' kernels
            # (largest copy first: the last layer's kernels are what nothing overlaps)
            cur = torch.cuda.current_stream()
            for h in sorted(host, key=lambda h: -(h["W"].numel() + h["X"].numel())):
                h["stream"].wait_stream(cur)
                with torch.cuda.stream(h["stream"]):
                    binding.quantize_layer_host_async(h["W"], h["X"], mode, n_outer=ROUNDS, init=binding.INIT_QUANTILE,
                                                      T01_host=h["T01"], T01_bf16_host=h["Tb"], scales_host=h["sc"],
                                                      tensor_scale_host=h["ts"], codes_host=h["codes"],
                                                      err_out_host=h["err"], status_host=h["status"], ws=h["ws"])
            for h in host:
                cur.wait_stream(h["stream"])
            cur.synchronize()                                  # the step's results are on the host
            if any(int(h["status"].item()) for h in host):
                raise RuntimeError("device status is set")
        for _ in range(2):
            host_step()
        barrier()
        e0.record()
        for _ in range(args.steps):
            host_step()
        e1.record()
        barrier()
        ms_e2e = sharding.max_over_ranks(e0.elapsed_time(e1), dev) / args.steps
        h2d = sum(h["W"].numel() * 2 + h["X"].numel() * 2 for h in host)
        d2h = sum(h["codes"].numel() + h["sc"].numel() + 128 + 64 + 4 + 16 + 4 for h in host)
        e2e = {"value": sharding.job_throughput(weights_per_step, ROUNDS, ms_e2e, world), "unit": UNIT,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "ms_per_step": ms_e2e}
    except Exception as ex:                                   # report, never hide
        e2e = {"value": None, "unit": UNIT, "error": repr(ex)}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, cores, sample, dt = cpu_baseline_sample(layers)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample, "seconds": dt}

    # the metric's second half: wall time of the whole decoder stacks (configurations 3 and 4)
    stacks = {}
    if rank == 0 and world == 1 and names == LAYERS and not args.no_stacks:
        del Wd, Xd, outs
        host.clear()
        torch.cuda.empty_cache()
        for which in ("stack8b", "stack7b"):
            try:
                r = run_stack(args, which, emit=False)
                stacks[which] = {"wall_s": r["value"], "gweights_per_s_per_round": r["gweights_per_s_per_round"],
                                 "workload": r["config"]["workload"], "clocks": r["clocks"], "gpu_launches": r["gpu_launches"]}
            except Exception as ex:                           # report, never hide
                stacks[which] = {"wall_s": None, "error": repr(ex)}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
                "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f32", "data": "synthetic",
                "config": {"workload": CFG2_WORKLOAD
                           if names == LAYERS else "cfg2 SUBSET (not the benchmark workload): " + ",".join(names),
                           "weights_per_step": weights_per_step, "rounds": ROUNDS, "seed": "rank",
                           "l2": "inputs larger than L2: 0.27 GB of W and 0.27 GB of X per step, three layers in turn",
                           "timing": f"{REPEATS} repeats of the {args.steps}-step timed loop; the median repeat is reported",
                           "ms_per_step_repeats": [r[0] / args.steps for r in reps]},
                "roofline": roofline, "roofline_other": roofline_other, "cpu_baseline": cpu, "e2e": e2e,
                "gpu_launches": int(launches),
                "stack8b_wall_s": (stacks.get("stack8b") or {}).get("wall_s"),
                "stack7b_wall_s": (stacks.get("stack7b") or {}).get("wall_s"),
                "stacks": stacks,
                "clocks": clocks, "wall_s_per_step": ms_step * 1e-3}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
