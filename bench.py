#!/usr/bin/env python
"""Benchmark of the quantized-linear hot path (rotate-quantize + int8 tensor-core GEMM with a
dequantizing epilogue) on HunyuanVideo-shaped layers, one JSON line on stdout.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one pass of the whole path over every layer of the workload (for each layer:
dvdq_rotate_quantize then dvdq_qgemm, i.e. what dvdq_qlinear runs) on synthetic inputs that
are already resident in HBM.  With N > 1 (torchrun, one rank per GPU) every rank runs the
same per-GPU work on its own seeded tokens, there is no data-path collective, and the value
is the aggregate over ranks divided by the slowest rank's time (weak scaling).

--impl reference times the CPU oracle (the only other implementation of this path that
exists) on a bounded token sample of the same workload.
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

import torch  # noqa: E402

METRIC = "W4A4/W4A6 qlinear throughput (rotate-quantize + int8 tcgen05 GEMM + dequant), TOPS = 2*M*N*K / time"
NOMINAL_INT8_TOPS = 4500.0
INT8_OVER_BF16 = 2.0           # nominal dense ratio, int8 : bf16
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0  # burst; about 1400 sustained


# ------------------------------------------------------------------ helpers

def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, power, reasons = [], None, [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax = float(parts[1])
                power.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": smax,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def layer_ops(M, layer):
    return 2.0 * M * layer.N * layer.K


def rq_bytes(M, layer, scale_group=0, container=0):
    """Algorithmic HBM bytes of rotate-quantize: bf16 row in, codes as stored + scales + code sums out."""
    per_token = layer.K // scale_group if scale_group else 1
    return M * (2.0 * layer.K + layer.K * (container or layer.bits) / 8.0 + 8.0 * per_token)


# ------------------------------------------------------------------ the CPU oracle leg

def oracle_sample(wl, tokens, steps=1, warmup=0, scale_group=0):
    """Times the CPU oracle, as it stands, on `tokens` tokens of every layer of the workload
    (rotation + quantizer + integer GEMM + epilogue; weight preparation is offline and not
    timed).  Returns (seconds per step, ops per step, threads)."""
    import numpy as np
    from oracle import dvdq_oracle as orc
    from paper_2505_18663_b200 import workloads as W

    def bits_of(t):
        return t.contiguous().view(torch.int16).numpy().view(np.uint16)

    prepared = []
    for i, layer in enumerate(wl.layers):
        x = W.make_activations(wl, layer.K, M=tokens)
        u, d, z = W.make_weight_codes(layer, seed=i)
        prepared.append((layer, bits_of(x), u.numpy(), d.numpy(), z.numpy()))
    ops = sum(layer_ops(tokens, l) for l in wl.layers)

    def one_step():
        for layer, xb, u, d, z in prepared:
            if scale_group:
                orc.qlinear_grouped(xb, u, d, z, layer.rot_block, layer.bits, scale_group, None, layer.act)
            else:
                orc.qlinear(xb, u, d, z, layer.rot_block, layer.bits, None, layer.act)

    for _ in range(warmup):
        one_step()
    t0 = time.perf_counter()
    for _ in range(steps):
        one_step()
    dt = (time.perf_counter() - t0) / steps
    return dt, ops, orc.num_threads()


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    tokens = args.ref_tokens
    dt, ops, threads = oracle_sample(wl, tokens, steps=args.steps, warmup=min(args.warmup, 1), scale_group=args.scale_group)
    value = ops / dt / 1e12
    sample = f"{tokens} tokens of each of the {len(wl.layers)} layers of '{wl.name}' per step (full K and N)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TOPS", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(wl, args),
        "cpu_baseline": {"value": value, "unit": "TOPS", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def config_of(wl, args):
    return {"workload": f"{wl.name}: M={wl.M} tokens, layers K->N " + ", ".join(
                f"{l.K}->{l.N} A{l.bits} B{l.rot_block}" for l in wl.layers),
            "weights": "4-bit per-output-channel codes (random, Gaussian-shaped)",
            "l2_policy": "inputs larger than L2 (every layer streams >= 400 MB)",
            "act_codes": ("one int8 per code" if args.container else "packed, b bits per code"),
            "act_scales": (f"one per token and block of {args.scale_group} channels" if args.scale_group else "one per token"),
            "parallelism": f"dp{args.gpus} (token-sharded replicas, no collective)"}


# ------------------------------------------------------------------ the CUDA leg

def run_cuda(args, wl):
    from paper_2505_18663_b200 import binding as B
    from paper_2505_18663_b200 import dist as D
    from paper_2505_18663_b200 import workloads as W

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    B.load()
    M = wl.M

    # ---- resident inputs (per rank: its own seeded tokens)
    xs = {}
    for layer in wl.layers:
        if layer.K not in xs:
            xs[layer.K] = W.make_activations(wl, layer.K, device=dev, salt=rank)
    layers = []
    for i, layer in enumerate(wl.layers):
        u, d, z = W.make_weight_codes(layer, seed=i, device=dev)
        blob = torch.empty(B.dvdq_weight_blob_bytes(layer.N, layer.K), dtype=torch.uint8, device=dev)
        w = B.dvdq_pack_weights(u, d, z, layer.rot_block, blob)
        del u
        q = B.ActQuant(layer.bits, layer.rot_block, args.scale_group, args.container)
        codes = torch.empty(B.dvdq_act_codes_bytes_q(M, layer.K, q), dtype=torch.uint8, device=dev)
        n_scales = B.dvdq_act_scales_count(M, layer.K, q)
        if n_scales == 0:
            raise SystemExit(f"layer {layer.K}->{layer.N}: activation quantizer options not supported")
        scales = torch.empty(n_scales, dtype=torch.float32, device=dev)
        sums = torch.empty(n_scales, dtype=torch.int32, device=dev)
        Y = torch.empty(M, layer.N, dtype=torch.bfloat16, device=dev)
        bias = W.make_bias(wl, layer, device=dev)
        layers.append(dict(layer=layer, w=w, blob=blob, q=q, codes=codes, scales=scales, sums=sums, Y=Y, bias=bias))
    torch.cuda.synchronize()

    def step(events=None):
        for li, L in enumerate(layers):
            layer = L["layer"]
            if events is not None:
                events[li][0].record()
            B.dvdq_rotate_quantize(xs[layer.K], L["q"], L["codes"], L["scales"], L["sums"])
            if events is not None:
                events[li][1].record()
            B.dvdq_qgemm(L["codes"], L["scales"], L["sums"], M, L["q"], L["w"], L["bias"], layer.act, L["Y"])
            if events is not None:
                events[li][2].record()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    status, detail = B.dvdq_last_device_status()
    if status != B.OK:
        raise SystemExit(f"device status {status} ({B.status_string(status)}), wait id {detail}")

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ev = [[[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in layers] for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_begin.record()
    for s in range(args.steps):
        step(ev[s])
    t_end.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    elapsed_ms = D.max_over_ranks(t_begin.elapsed_time(t_end), dist, dev)
    status, detail = B.dvdq_last_device_status()
    if status != B.OK:
        raise SystemExit(f"device status {status} ({B.status_string(status)}), wait id {detail}")

    ms_per_step = elapsed_ms / args.steps
    ops_per_step = sum(layer_ops(M, L["layer"]) for L in layers)
    value = D.aggregate_rate(ops_per_step, ms_per_step, world) / 1e12

    # ---- per-kernel durations from the events of the timed region (this rank)
    rq_ms = [sum(ev[s][li][0].elapsed_time(ev[s][li][1]) for s in range(args.steps)) / args.steps for li in range(len(layers))]
    gm_ms = [sum(ev[s][li][1].elapsed_time(ev[s][li][2]) for s in range(args.steps)) / args.steps for li in range(len(layers))]
    peaks = load_peaks()
    int8_peak = peaks["bf16_tflops_sustained"] * INT8_OVER_BF16
    gemm_ops = sum(layer_ops(M, L["layer"]) for L in layers)
    gemm_tops = gemm_ops / (sum(gm_ms) * 1e-3) / 1e12
    rq_total_bytes = sum(rq_bytes(M, L["layer"], args.scale_group, args.container) for L in layers)
    rq_gbs = rq_total_bytes / (sum(rq_ms) * 1e-3) / 1e9
    stages = []
    for li, L in enumerate(layers):
        layer = L["layer"]
        stages.append({"layer": f"{layer.K}->{layer.N} A{layer.bits}",
                       "rq_ms": rq_ms[li], "rq_gbs": rq_bytes(M, layer, args.scale_group, args.container) / (rq_ms[li] * 1e-3) / 1e9,
                       "qgemm_ms": gm_ms[li], "qgemm_tops": layer_ops(M, layer) / (gm_ms[li] * 1e-3) / 1e12})

    # ---- rotate-quantize on its own (no GEMM between the launches, so no GEMM drawing the power budget down)
    n_alone = 0 if args.no_alone else max(5, args.steps // 5)
    ev_alone = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in layers] for _ in range(n_alone)]
    for it in range(3 + n_alone if n_alone else 0):
        for li, L in enumerate(layers):
            layer = L["layer"]
            if it >= 3:
                ev_alone[it - 3][li][0].record()
            B.dvdq_rotate_quantize(xs[layer.K], L["q"], L["codes"], L["scales"], L["sums"])
            if it >= 3:
                ev_alone[it - 3][li][1].record()
    torch.cuda.synchronize()
    rq_alone = None
    if n_alone:
        rq_alone_ms = sum(a.elapsed_time(b) for row in ev_alone for a, b in row) / n_alone
        rq_alone_gbs = rq_total_bytes / (rq_alone_ms * 1e-3) / 1e9
        rq_alone = {"achieved": rq_alone_gbs, "frac": rq_alone_gbs / load_peaks()["hbm_gbs"], "steps": n_alone,
                    "note": "the same launches without the GEMMs between them"}

    # ---- the same step with the codes packed b bits each (container 0), for the record: fewer steps
    packed = None
    if args.container != 0 and not args.no_packed and world == 1:
        packed = run_packed_leg(args, wl, layers, xs, dev, B, M)

    # ---- end to end through dvdq_qlinear with HOST buffers (pinned), copies inside the timed region
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, wl, layers, xs, dev, B, dist, world)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # the ncu counters were taken on the default workload (hunyuan, its own bit widths, per-token scales)
    captured = wl.name == "hunyuan" and wl.M == 65536 and args.bits == 0 and args.scale_group == 0 and args.container == 8
    line = {
        "metric": METRIC, "value": value, "unit": "TOPS", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "i8", "data": "synthetic", "config": config_of(wl, args),
        "roofline": {"kernel": ("qgemm_ss_kernel" if args.container == 8 and args.scale_group == 0 else "qgemm_kernel") + " (tcgen05.mma kind::i8)", "bound": "tensor", "achieved": gemm_tops,
                     "peak": int8_peak, "unit": "TOPS", "frac": gemm_tops / int8_peak,
                     "peak_source": f"{peaks['source']}: bf16_tflops_sustained x {INT8_OVER_BF16} (nominal int8:bf16)",
                     "frac_of_nominal_4500": gemm_tops / NOMINAL_INT8_TOPS,
                     "avg_launch_ms": sum(gm_ms) / len(gm_ms), "traffic": QGEMM_DRAM_TRAFFIC_PER_LAUNCH if captured else None},
        "roofline_rotate_quantize": {"kernel": "rq_kernel", "bound": "hbm", "achieved": rq_gbs,
                                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": rq_gbs / peaks["hbm_gbs"],
                                     "peak_source": peaks["source"], "frac_of_nominal_8000": rq_gbs / 8000.0,
                                     "avg_launch_ms": sum(rq_ms) / len(rq_ms), "traffic": RQ_DRAM_TRAFFIC_PER_LAUNCH if captured else None,
                                     "alone": rq_alone},
        "stages": stages,
        "packed_codes": packed,
        "e2e": e2e,
        "gpu_launches": 2 * len(layers) * args.steps,
        "clocks": clocks,
    }
    if not args.no_cpu_baseline and world == 1:
        dt, ops, threads = oracle_sample(wl, args.ref_tokens, scale_group=args.scale_group)
        line["cpu_baseline"] = {"value": ops / dt / 1e12, "unit": "TOPS", "cores": threads, "kind": "oracle",
                                "sample": f"{args.ref_tokens} tokens of each layer of '{wl.name}' (full K and N), {dt:.1f} s"}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# DRAM bytes (read + write) per launch from the ncu captures summarised under profiles/; None
# until a capture of the corresponding kernel exists.
QGEMM_DRAM_TRAFFIC_PER_LAUNCH = 1.15e9   # bytes: 16384-token capture x 4 (traffic grows with M), mean of the 4 layers
RQ_DRAM_TRAFFIC_PER_LAUNCH = 0.94e9


def run_packed_leg(args, wl, layers, xs, dev, B, M):
    """The step with activation codes packed b bits each (the layout the GEMM widens in shared and
    tensor memory), timed on max(5, steps / 5) steps after 3 warm-up steps.  Same inputs, same outputs."""
    packed_layers = []
    for L in layers:
        layer = L["layer"]
        q = B.ActQuant(layer.bits, layer.rot_block, args.scale_group, 0)
        codes = torch.empty(B.dvdq_act_codes_bytes_q(M, layer.K, q), dtype=torch.uint8, device=dev)
        packed_layers.append((layer, q, codes, L))
    n_steps = max(5, args.steps // 5)
    ev = [[[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in packed_layers] for _ in range(n_steps)]

    def step(events=None):
        for li, (layer, q, codes, L) in enumerate(packed_layers):
            if events is not None:
                events[li][0].record()
            B.dvdq_rotate_quantize(xs[layer.K], q, codes, L["scales"], L["sums"])
            if events is not None:
                events[li][1].record()
            B.dvdq_qgemm(codes, L["scales"], L["sums"], M, q, L["w"], L["bias"], layer.act, L["Y"])
            if events is not None:
                events[li][2].record()

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for s in range(n_steps):
        step(ev[s])
    t1.record()
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / n_steps
    rq_ms = sum(ev[s][li][0].elapsed_time(ev[s][li][1]) for s in range(n_steps) for li in range(len(packed_layers))) / n_steps
    gm_ms = sum(ev[s][li][1].elapsed_time(ev[s][li][2]) for s in range(n_steps) for li in range(len(packed_layers))) / n_steps
    ops = sum(layer_ops(M, l) for l, _, _, _ in packed_layers)
    nbytes = sum(rq_bytes(M, l, args.scale_group, 0) for l, _, _, _ in packed_layers)
    return {"value": ops / (ms * 1e-3) / 1e12, "unit": "TOPS", "ms_per_step": ms, "steps": n_steps,
            "qgemm_tops": ops / (gm_ms * 1e-3) / 1e12, "rq_gbs": nbytes / (rq_ms * 1e-3) / 1e9}


def run_e2e(args, wl, layers, xs, dev, B, dist, world):
    """Same metric through the user-facing call dvdq_qlinear, with the layer input copied from
    pinned host memory and the layer output copied back to pinned host memory inside every step.
    Three streams (copy-in, compute, copy-out) and two device input buffers let the PCIe copies of
    neighbouring layers overlap the kernels; every byte still crosses the bus inside the timed region."""
    M = wl.M
    maxK = max(L["layer"].K for L in layers)
    maxN = max(L["layer"].N for L in layers)
    host_x = {K: x.to("cpu").pin_memory() for K, x in xs.items()}
    host_y = [torch.empty(M, maxN, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    dev_x = [torch.empty(M, maxK, dtype=torch.bfloat16, device=dev) for _ in range(2)]
    ws = torch.empty(max(B.dvdq_qlinear_workspace_bytes(M, L["layer"].K, L["q"]) for L in layers), dtype=torch.uint8, device=dev)
    h2d = sum(M * L["layer"].K * 2 for L in layers)
    d2h = sum(M * L["layer"].N * 2 for L in layers)
    s_in, s_run, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    n = len(layers)
    in_done = [torch.cuda.Event() for _ in range(2)]     # dev_x[b] filled
    in_free = [torch.cuda.Event() for _ in range(2)]     # dev_x[b] consumed by its layer
    run_done = [torch.cuda.Event() for _ in range(n)]    # Y of layer i written
    out_done_layer = [torch.cuda.Event() for _ in range(n)]  # Y of layer i copied out
    counter = [0]

    def step():
        for li, L in enumerate(layers):
            layer = L["layer"]
            c = counter[0]
            b = c & 1
            xd = dev_x[b].view(-1)[: M * layer.K].view(M, layer.K)
            with torch.cuda.stream(s_in):
                if c >= 2:
                    s_in.wait_event(in_free[b])
                xd.copy_(host_x[layer.K], non_blocking=True)
                in_done[b].record(s_in)
            with torch.cuda.stream(s_run):
                s_run.wait_event(in_done[b])
                if c >= n:
                    s_run.wait_event(out_done_layer[li])  # the previous step's copy-out of this layer's Y
                B.dvdq_qlinear(xd, L["q"], L["w"], L["bias"], layer.act, L["Y"], ws, stream=s_run)
                in_free[b].record(s_run)
                run_done[li].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(run_done[li])
                host_y[b].view(-1)[: M * layer.N].view(M, layer.N).copy_(L["Y"], non_blocking=True)
                out_done_layer[li].record(s_out)
            counter[0] = c + 1

    steps = max(1, min(args.steps, 3))
    step()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cur = torch.cuda.current_stream()
    t0.record(cur)
    for s in (s_in, s_run, s_out):
        s.wait_event(t0)
    for _ in range(steps):
        step()
    for s in (s_in, s_run, s_out):
        ev = torch.cuda.Event()
        ev.record(s)
        cur.wait_event(ev)
    t1.record(cur)
    torch.cuda.synchronize()
    from paper_2505_18663_b200 import dist as D
    ms = D.max_over_ranks(t0.elapsed_time(t1) / steps, dist, dev)
    ops = sum(layer_ops(M, L["layer"]) for L in layers)
    return {"value": world * ops / (ms * 1e-3) / 1e12, "unit": "TOPS", "ms_per_step": ms, "steps": steps,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "api": "dvdq_qlinear, pinned host buffers, copy-in / compute / copy-out streams"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="hunyuan")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--ref-tokens", type=int, default=384, help="token sample timed on the CPU oracle")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--tokens", type=int, default=0, help="override the workload's token count (profiling runs)")
    ap.add_argument("--container", type=int, default=8,
                    help="8: one int8 per activation code (default, the faster GEMM); 0: codes packed b bits each")
    ap.add_argument("--no-packed", action="store_true", help="skip the extra leg that times the packed layout")
    ap.add_argument("--no-alone", action="store_true", help="skip the extra leg that times rotate-quantize on its own")
    ap.add_argument("--scale-group", type=int, default=0,
                    help="0: one activation scale per token; 1024: one per token and block of 1024 channels")
    ap.add_argument("--bits", type=int, default=0, help="override the activation bit width of every layer (4, 6 or 8)")
    args = ap.parse_args()
    from paper_2505_18663_b200 import workloads as W
    wl = W.WORKLOADS[args.workload]
    if args.tokens > 0:
        import dataclasses
        wl = dataclasses.replace(wl, M=args.tokens)
    if args.bits > 0:
        import dataclasses
        wl = dataclasses.replace(wl, layers=tuple(dataclasses.replace(l, bits=args.bits) for l in wl.layers))
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_cuda(args, wl)


if __name__ == "__main__":
    main()
