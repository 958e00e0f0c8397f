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
KERNELS_PER_LAYER = 2 + 3 + 6 + 1 + 1 + 2 + 1   # act_stats, scales, init, fit rounds (one launch), export, pack, dequant


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def measured_traffic_per_weight():
    """DRAM bytes per weight and round of the fit-rounds kernel, from the line
    `dram_bytes_per_weight_round = X` of the committed ncu summary (None if absent)."""
    p = os.path.join(ROOT, "profiles", "fit_rounds_cfg2_gate_proj.md")
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
    """Reference arm = the CPU oracle on a bounded sample per step."""
    if rank != 0:
        return
    layers = [__import__("paper_2605_08692_b200.synth", fromlist=["x"]).config2_layer("q_proj", seed=0, rows=1024, tokens=256)]
    vals = []
    for i in range(args.warmup + args.steps):
        v, cores, sample, dt = cpu_baseline_sample(layers, rounds=ROUNDS, rows=1024)
        if i >= args.warmup:
            vals.append((v, dt))
    value = float(np.mean([v for v, _ in vals]))
    ms = float(np.mean([d for _, d in vals]) * 1e3)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "cfg2 Llama-3-8B-shaped linears, NVFP4 g16, 20 rounds (bounded sample per step)"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


STACKS = {
    # name: (decoder layers, hidden, kv width, intermediate, mode, tokens, rounds)
    "stack8b": (32, 4096, 1024, 14336, 0, 16384, 20),     # Llama-3-8B-shaped, INT4 g128
    "stack7b": (28, 3584, 512, 18944, 1, 16384, 20),      # Qwen2.5-7B-shaped, NVFP4 g16
}


def run_stack(args, which):
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
    Iv = {k: torch.empty(x.shape[1], dtype=torch.float32, device=dev) for k, x in X.items()}
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    def decoder_layer():
        for k, x in X.items():
            binding.act_stats(x, Iv[k], out["down" if k == "down" else "q"]["ws"], dev_status=status)
        for n, N, K, xin in lin:
            o = out[n]
            binding.fit_layer(Ws[n], mode, I=Iv[xin], n_outer=rounds, n_inner=n_inner, init=binding.INIT_QUANTILE,
                              T01=o["T01"], scales=o["scales"], tensor_scale=o["ts"], ws=o["ws"], dev_status=status,
                              sel_group=sel)
            binding.pack(Ws[n], mode, I=Iv[xin], T01=o["T01"], T01_bf16=o["Tb"], scales=o["scales"],
                         tensor_scale=o["ts"], codes=o["codes"], ws=o["ws"], err_out=o["err"], sel_group=sel,
                         sigma_bits=o["bits"])

    for _ in range(2):
        decoder_layer()
    torch.cuda.synchronize()
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
                                   f"n_outer {rounds}, n_inner {n_inner}; act_stats + scales + init + rounds + pack",
                       "linears": 7 * L, "weights": wl * L, "rounds": rounds, "n_inner": n_inner},
            "gweights_per_s_per_round": wl * L * rounds * n_inner / wall / 1e9, "clocks": clocks}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
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

    def step():
        for W, X, o in zip(Wd, Xd, outs):
            binding.act_stats(X, o["I"], o["ws"], dev_status=status)
            binding.fit_layer(W, mode, I=o["I"], n_outer=ROUNDS, init=binding.INIT_QUANTILE, T01=o["T01"],
                              scales=o["scales"], tensor_scale=o["ts"], ws=o["ws"], dev_status=status)
            binding.pack(W, mode, I=o["I"], T01=o["T01"], T01_bf16=o["Tb"], scales=o["scales"], tensor_scale=o["ts"],
                         codes=o["codes"], ws=o["ws"], err_out=o["err"])
            binding.dequant(o["codes"], o["scales"], o["ts"], o["Tb"], mode, o["What"])

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
    binding.timing_begin(args.steps * len(layers))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    round_ms = binding.timing_end(args.steps * len(layers))      # one entry per fit launch (all rounds of a layer)
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
    ms_total = sharding.max_over_ranks(ms_total, dev)
    ms_step = ms_total / args.steps
    value = sharding.job_throughput(weights_per_step, ROUNDS, ms_step, world)

    # roofline of the dominant kernel: algorithmic bytes of every timed fit-round launch / its device time
    per_launch_w = []
    for _ in range(args.steps):
        for (N, K) in shapes:
            per_launch_w += [N * K * ROUNDS]
    bytes_alg = sum(per_launch_w[:len(round_ms)]) * BYTES_PER_WEIGHT
    fit_ms = float(sum(round_ms))
    achieved = bytes_alg / (fit_ms * 1e-3) / 1e9 if fit_ms > 0 else 0.0
    peak, peak_kind = peaks()
    tpw = measured_traffic_per_weight()
    roofline = {"kernel": "fit_rounds_kernel (one launch = the 20 k-means rounds of a layer)", "bound": "hbm", "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "peak_source": f"of {peak_kind}",
                "traffic": None if tpw is None else tpw * float(np.mean(per_launch_w)),
                "algorithmic_bytes_per_launch": float(np.mean(per_launch_w)) * BYTES_PER_WEIGHT,
                "avg_launch_ms": fit_ms / max(len(round_ms), 1),
                "fit_share_of_step": fit_ms / ms_total if ms_total > 0 else None,
                "gweights_per_s_kernel": sum(per_launch_w[:len(round_ms)]) / (fit_ms * 1e-3) / 1e9 if fit_ms else 0.0}

    # end to end through the host-buffer entry point (pinned host memory in and out)
    e2e = None
    try:
        host = []
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

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
                "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f32", "data": "synthetic",
                "config": {"workload": ("cfg2: Llama-3-8B-shaped q_proj 4096x4096, gate_proj 14336x4096, down_proj "
                                        "4096x14336; NVFP4 g16 E4M3 scales; X 4096 tokens; quantile init; 20 rounds; "
                                        "step = act_stats + scales + init + 20 fit rounds + pack + dequant per layer")
                           if names == LAYERS else "cfg2 SUBSET (not the benchmark workload): " + ",".join(names),
                           "weights_per_step": weights_per_step, "rounds": ROUNDS, "seed": "rank",
                           "l2": "inputs larger than L2: 0.27 GB of W and 0.27 GB of X per step, three layers in turn"},
                "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
                "gpu_launches": KERNELS_PER_LAYER * len(layers) * args.steps,
                "clocks": clocks, "wall_s_per_step": ms_step * 1e-3}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
