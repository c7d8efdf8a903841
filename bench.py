#!/usr/bin/env python
"""Benchmark of the quantized-linear hot path (rotate-quantize + int8 tensor-core GEMM with a
dequantizing epilogue) on HunyuanVideo-shaped layers, one JSON line on stdout.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME|all] [--impl reference]

A step is one pass of the whole path over every layer of the workload (for each layer:
dvdq_rotate_quantize then dvdq_qgemm, i.e. what dvdq_qlinear runs) on synthetic inputs that
are already resident in HBM.  The headline keeps the activation codes packed b bits each (the
GEMM widens them); the same step with one int8 per code is timed beside it (`other_layout`).
Rooflines: the GEMM against the int8 tensor-pipe ceiling measured in the same run (an issue loop
on resident operands), rotate-quantize against the measured copy rate on its ALGORITHMIC bytes.  With N > 1 (torchrun, one rank per GPU) every rank runs the
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
NOMINAL_HBM_GBS = 8000.0
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
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20"],
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


def rq_algorithmic_bytes(M, layer, scale_group=0):
    """Algorithmic HBM bytes of rotate-quantize per launch: the bf16 row in, b-bit codes and one
    scale + one code sum per scale group out: 2K + K b / 8 + 8 per token and group, whatever
    container the codes are kept in."""
    per_token = layer.K // scale_group if scale_group else 1
    return M * (2.0 * layer.K + layer.K * layer.bits / 8.0 + 8.0 * per_token)


def rq_stored_bytes(M, layer, scale_group=0, container=0):
    """Bytes the kernel actually moves: as above with the codes at their stored width."""
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
            "fused": bool(getattr(args, "fuse", False) and wl.chain),
            "parallelism": f"dp{args.gpus} (token-sharded replicas, no collective)"}


# ------------------------------------------------------------------ the CUDA leg

# DRAM bytes (read + write) per launch from the ncu captures summarised under profiles/, by code
# layout (container_bits); None where no capture of that kernel in its present form exists.
# (16384-token capture x 4: traffic grows with M; mean of the four launches of a step; the GEMM with
# its weight operand written before every launch, the default)
QGEMM_DRAM_TRAFFIC_PER_LAUNCH = {0: 1.17e9, 8: 1.52e9}
RQ_DRAM_TRAFFIC_PER_LAUNCH = {0: 0.82e9, 8: 0.94e9}


class Leg:
    """One code layout of the workload: its buffers, and the step that launches rotate-quantize
    and the GEMM for every layer (what dvdq_qlinear runs), optionally with CUDA events around
    every launch."""

    def __init__(self, B, W, wl, args, container, dev, rank, shared=None, fuse=False):
        self.B, self.wl, self.container, self.scale_group = B, wl, container, args.scale_group
        self.fuse = fuse and wl.chain   # every layer but the last writes the next layer's codes instead of bf16
        if self.fuse and (container != 8 or args.scale_group != 0):
            raise SystemExit("--fuse needs --container 8 and per-token scales on the first layer")
        M = self.M = wl.M
        if shared is None:
            xs = {}
            first = wl.layers[0]
            for layer in (wl.layers[:1] if wl.chain else wl.layers):
                if layer.K not in xs:
                    xs[layer.K] = W.make_activations(wl, layer.K, device=dev, salt=rank)
            weights = []
            for i, layer in enumerate(wl.layers):
                u, d, z = W.make_weight_codes(layer, seed=i, device=dev)
                blob = torch.empty(B.dvdq_weight_blob_bytes(layer.N, layer.K), dtype=torch.uint8, device=dev)
                rot = 256 if (self.fuse and i > 0) else layer.rot_block   # recorded in the blob: what the activations are rotated with
                weights.append((B.dvdq_pack_weights(u, d, z, rot, blob), blob, W.make_bias(wl, layer, device=dev)))
                del u
            Ys = [torch.empty(M, layer.N, dtype=torch.bfloat16, device=dev) for layer in wl.layers]
            # one scratch area for the int8 weight operand of whichever layer runs next (rewritten before every GEMM)
            scratch = torch.empty(max(layer.N * layer.K for layer in wl.layers), dtype=torch.uint8, device=dev)
            shared = dict(xs=xs, weights=weights, Ys=Ys, scratch=scratch)
        self.shared = shared
        # where the GEMM's int8 weight operand comes from: widened inside the GEMM by every tile ("tile"), written
        # into the scratch area before every GEMM launch ("launch", inside the timed region), or kept ("resident")
        self.operand = args.weight_operand
        self.layers = []
        for i, layer in enumerate(wl.layers):
            q = B.ActQuant(layer.bits, layer.rot_block, args.scale_group, container)
            if self.fuse and i > 0:
                q = B.ActQuant(layer.bits, 256, 256, 8)   # what the fused epilogue of the layer before produces
            n_scales = B.dvdq_act_scales_count(M, layer.K, q)
            if n_scales == 0:
                raise SystemExit(f"layer {layer.K}->{layer.N}: activation quantizer options not supported")
            # in a chain every layer but the first reads the previous layer's output
            x = shared["Ys"][i - 1] if (wl.chain and i > 0) else shared["xs"][layer.K]
            w, _, bias = shared["weights"][i]
            if self.operand == "resident":
                keep = torch.empty(layer.N * layer.K, dtype=torch.uint8, device=dev)
                w = B.dvdq_widen_weights(w, keep)
                self.kept = getattr(self, "kept", []) + [keep]
            self.layers.append(dict(layer=layer, q=q, x=x, w=w, bias=bias, Y=shared["Ys"][i],
                                    codes=torch.empty(B.dvdq_act_codes_bytes_q(M, layer.K, q), dtype=torch.uint8, device=dev),
                                    scales=torch.empty(n_scales, dtype=torch.float32, device=dev),
                                    sums=torch.empty(n_scales, dtype=torch.int32, device=dev)))

    def step(self, events=None, rq_only=False):
        B = self.B
        n = len(self.layers)
        for li, L in enumerate(self.layers):
            if events is not None:
                events[li][0].record()
            if not (self.fuse and li > 0):
                B.dvdq_rotate_quantize(L["x"], L["q"], L["codes"], L["scales"], L["sums"])
            if events is not None:
                events[li][1].record()
            if rq_only:
                continue
            w = L["w"]
            if self.operand == "launch":
                w = B.dvdq_widen_weights(w, self.shared["scratch"][:L["layer"].N * L["layer"].K])
            if self.fuse and li + 1 < n:
                nx = self.layers[li + 1]
                B.dvdq_qgemm_fused_rq(L["codes"], L["scales"], L["sums"], self.M, L["q"], w, L["bias"], L["layer"].act,
                                      nx["q"], nx["codes"], nx["scales"], nx["sums"])
            else:
                B.dvdq_qgemm(L["codes"], L["scales"], L["sums"], self.M, L["q"], w, L["bias"], L["layer"].act, L["Y"])
            if events is not None:
                events[li][2].record()

    def launches_per_step(self):
        return 2 * len(self.layers) - (len(self.layers) - 1 if self.fuse else 0) + (len(self.layers) if self.operand == "launch" else 0)

    def timed(self, steps, warmup, barrier, rq_only=False):
        """(ms per step, per-layer rq ms, per-layer GEMM ms) from CUDA events inside the timed region."""
        for _ in range(warmup):
            self.step(rq_only=rq_only)
        n = len(self.layers)
        ev = [[[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n)] for _ in range(steps)]
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0.record()
        for s in range(steps):
            self.step(ev[s], rq_only=rq_only)
        t1.record()
        barrier()
        rq_ms = [sum(ev[s][li][0].elapsed_time(ev[s][li][1]) for s in range(steps)) / steps for li in range(n)]
        gm_ms = [0.0] * n if rq_only else [sum(ev[s][li][1].elapsed_time(ev[s][li][2]) for s in range(steps)) / steps for li in range(n)]
        return t0.elapsed_time(t1) / steps, rq_ms, gm_ms


def measure_int8_ceiling(B, seconds, local_rank):
    """The int8 tensor-pipe ceiling of this GPU, now: the issue loop of dvdq_int8_mma_ceiling
    (resident operands, no loads, no epilogue) repeated for about `seconds`, with the SM clock
    sampled meanwhile."""
    B.dvdq_int8_mma_ceiling(2000)
    torch.cuda.synchronize()
    iters = 20000                        # about 5.5 ms per launch at the nominal rate
    n = max(3, min(400, int(seconds / 0.0055)))
    sampler = ClockSampler(local_rank)
    sampler.start()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    ops = 0
    for _ in range(n):
        ops += B.dvdq_int8_mma_ceiling(iters)
    t1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = t0.elapsed_time(t1)
    return {"tops": ops / (ms * 1e-3) / 1e12, "ms": ms, "launches": n, "sm_mhz": clocks.get("sm_mhz"),
            "reasons": clocks.get("reasons"), "what": "tcgen05.mma.cta_group::2.kind::i8 256x256x32 issue loop, operands resident in shared memory"}


def roofline_blocks(leg, ms_per_step, rq_ms, gm_ms, args, peaks, ceiling, timed_s):
    """The two roofline objects of a leg (GEMM: tensor-bound; rotate-quantize: HBM-bound) and its stages."""
    M, layers, sg, cont = leg.M, leg.layers, leg.scale_group, leg.container
    gemm_tops = sum(layer_ops(M, L["layer"]) for L in layers) / (sum(gm_ms) * 1e-3) / 1e12
    has_rq = [not (leg.fuse and li > 0) for li in range(len(layers))]   # fused: only the first layer launches rotate-quantize
    alg = sum(rq_algorithmic_bytes(M, L["layer"], sg) for L, h in zip(layers, has_rq) if h)
    stored = sum(rq_stored_bytes(M, L["layer"], sg, cont) for L, h in zip(layers, has_rq) if h)
    rq_ms = [t if h else 0.0 for t, h in zip(rq_ms, has_rq)]
    rq_gbs = alg / (sum(rq_ms) * 1e-3) / 1e9
    gemm_kernel = "qgemm_ss_kernel<8>" if cont == 8 else "qgemm_ss_kernel<4|6>"
    if sg or leg.fuse:
        gemm_kernel = "qgemm_fat_kernel"
    # without a ceiling measured in this run the GEMM is held against the nominal dense int8 rate
    peak = ceiling["tops"] if ceiling else NOMINAL_INT8_TOPS
    roof = {"kernel": gemm_kernel + " (tcgen05.mma kind::i8)", "bound": "tensor", "achieved": gemm_tops, "peak": peak, "unit": "TOPS",
            "frac": gemm_tops / peak,
            "peak_source": ("measured in this run: int8 issue-loop ceiling (dvdq_int8_mma_ceiling) at a median SM clock of "
                            f"{ceiling['sm_mhz']} MHz" if ceiling else "nominal dense int8 rate (no ceiling measured in this run)"),
            "frac_of_nominal_4500": gemm_tops / NOMINAL_INT8_TOPS,
            "frac_of_2x_bf16_burst": gemm_tops / (peaks["bf16_tflops"] * INT8_OVER_BF16),
            "frac_of_2x_bf16_sustained": gemm_tops / (peaks["bf16_tflops_sustained"] * INT8_OVER_BF16),
            "avg_launch_ms": sum(gm_ms) / len(gm_ms), "traffic": QGEMM_DRAM_TRAFFIC_PER_LAUNCH.get(cont) if args.default_workload else None}
    rq_roof = {"kernel": "rq_kernel", "bound": "hbm", "achieved": rq_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
               "frac": rq_gbs / peaks["hbm_gbs"], "peak_source": peaks["source"] + ": hbm_gbs (copy rate)",
               "frac_of_nominal_8000": rq_gbs / NOMINAL_HBM_GBS,
               "bytes": "algorithmic: 2K + K b/8 + 8 per token and scale group",
               "stored_bytes_gbs": stored / (sum(rq_ms) * 1e-3) / 1e9,
               "avg_launch_ms": sum(rq_ms) / sum(has_rq), "traffic": RQ_DRAM_TRAFFIC_PER_LAUNCH.get(cont) if args.default_workload else None}
    stages = []
    for li, L in enumerate(layers):
        layer = L["layer"]
        rq_g = rq_algorithmic_bytes(M, layer, sg) / (rq_ms[li] * 1e-3) / 1e9 if has_rq[li] else None
        stages.append({"layer": f"{layer.K}->{layer.N} A{layer.bits} B{L['q'].rot_block}" + (f" G{L['q'].scale_group}" if L['q'].scale_group else "")
                       + (" gelu" if layer.act else "") + (" bias" if layer.bias else "")
                       + (" [epilogue = next layer's rotate-quantize]" if leg.fuse and li + 1 < len(layers) else "")
                       + (" [codes from the previous GEMM's epilogue]" if not has_rq[li] else ""),
                       "rq_ms": rq_ms[li] if has_rq[li] else None, "rq_gbs": rq_g,
                       "rq_frac_of_hbm": rq_g / peaks["hbm_gbs"] if has_rq[li] else None,
                       "qgemm_ms": gm_ms[li], "qgemm_tops": layer_ops(M, layer) / (gm_ms[li] * 1e-3) / 1e12,
                       "qgemm_frac_of_peak": layer_ops(M, layer) / (gm_ms[li] * 1e-3) / 1e12 / peak})
    return roof, rq_roof, stages


def run_workload(args, wl, B, W, D, dist, dev, rank, local_rank, world, peaks, full, ceiling=None):
    """Times one workload; `full` adds the legs of the headline line (other layout, alone, ceiling, e2e, oracle)."""
    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def check_status():
        status, detail = B.dvdq_last_device_status()
        if status != B.OK:
            raise SystemExit(f"device status {status} ({B.status_string(status)}), wait id {detail}")

    leg = Leg(B, W, wl, args, args.container, dev, rank, fuse=args.fuse)
    M = wl.M
    warm = max(args.warmup, 3)
    leg.timed(1, warm - 1, barrier)   # warm-up (and first-use set-up) outside the sampled region
    check_status()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms_local, rq_ms, gm_ms = leg.timed(args.steps, 0, barrier)
    clocks = sampler.stop() if rank == 0 else None
    ms_per_step = D.max_over_ranks(ms_local, dist, dev)
    check_status()
    ops_per_step = sum(layer_ops(M, L["layer"]) for L in leg.layers)
    value = D.aggregate_rate(ops_per_step, ms_per_step, world) / 1e12
    timed_s = ms_per_step * args.steps * 1e-3

    if full and not args.no_ceiling:
        ceiling = measure_int8_ceiling(B, min(2.0, max(0.1, timed_s)), local_rank)
        check_status()
    roof, rq_roof, stages = roofline_blocks(leg, ms_per_step, rq_ms, gm_ms, args, peaks, ceiling, timed_s)

    out = {"value": value, "ms_per_step": ms_per_step, "roofline": roof, "roofline_rotate_quantize": rq_roof, "stages": stages,
           "clocks": clocks, "gpu_launches": leg.launches_per_step() * args.steps, "ceiling": ceiling, "leg": leg}
    def other_layout_leg():
        other = 8 if args.container == 0 else 0
        leg2 = Leg(B, W, wl, args, other, dev, rank, shared=leg.shared)
        n2 = max(5, min(args.steps, 50))
        ms2, rq2, gm2 = leg2.timed(n2, 3, barrier)
        check_status()
        r2, rr2, st2 = roofline_blocks(leg2, ms2, rq2, gm2, args, peaks, ceiling, ms2 * n2 * 1e-3)
        return {"act_codes": "one int8 per code" if other == 8 else "packed, b bits per code",
                "value": ops_per_step / (ms2 * 1e-3) / 1e12, "unit": "TOPS", "ms_per_step": ms2, "steps": n2,
                "roofline": r2, "roofline_rotate_quantize": rr2, "stages": st2}

    if not full:
        if not args.no_other_layout and world == 1 and not leg.fuse:
            out["other_layout"] = other_layout_leg()
        return out

    # ---- rotate-quantize on its own (no GEMM between the launches drawing the power budget down)
    if not args.no_alone:
        n_alone = max(5, args.steps // 2)
        _, rq_alone_ms, _ = leg.timed(n_alone, 3, barrier, rq_only=True)
        alg = sum(rq_algorithmic_bytes(M, L["layer"], args.scale_group) for li, L in enumerate(leg.layers) if not (leg.fuse and li > 0))
        g = alg / (sum(t for li, t in enumerate(rq_alone_ms) if not (leg.fuse and li > 0)) * 1e-3) / 1e9
        rq_roof["alone"] = {"achieved": g, "frac": g / peaks["hbm_gbs"], "frac_of_nominal_8000": g / NOMINAL_HBM_GBS, "steps": n_alone,
                            "note": "the same launches without the GEMMs between them"}

    # ---- the same step with the other code layout, as a full block of its own
    if not args.no_other_layout and world == 1 and not leg.fuse:
        out["other_layout"] = other_layout_leg()
    return out


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
    peaks = load_peaks()
    args.default_workload = (wl.name == "hunyuan" and wl.M == 65536 and args.bits == 0 and args.scale_group == 0
                             and args.weight_operand == "launch")

    res = run_workload(args, wl, B, W, D, dist, dev, rank, local_rank, world, peaks, full=True)
    leg = res.pop("leg")

    # ---- end to end through dvdq_qlinear with HOST buffers (pinned), copies inside the timed region
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, wl, leg, dev, B, dist, world)
    del leg

    # ---- the other configurations, one after the other (per-layer stages and rooflines only)
    extra = None
    if args.all_workloads and world == 1:
        import dataclasses
        extra = {}
        todo = [(n, w, 0) for n, w in W.WORKLOADS.items() if n not in (wl.name, "tiny")]
        # the HunyuanVideo shapes at both bit widths (the headline runs the seeded 25 % mask)
        todo += [("hunyuan_all_A4", W.WORKLOADS["hunyuan"], 4), ("hunyuan_all_A6", W.WORKLOADS["hunyuan"], 6)]
        # the K = 12288 layer with rotation blocks of 4096 channels (blocks that span four warps of the transform)
        todo += [("hunyuan_B4096_for_K12288", W.WORKLOADS["hunyuan"], -4096)]
        for name, w2, bits in todo:
            if bits > 0:
                w2 = dataclasses.replace(w2, layers=tuple(dataclasses.replace(l, bits=bits) for l in w2.layers))
            elif bits < 0:
                w2 = dataclasses.replace(w2, layers=tuple(dataclasses.replace(l, rot_block=-bits) if l.K % -bits == 0 else l for l in w2.layers))
            torch.cuda.empty_cache()
            r = run_workload(args, w2, B, W, D, dist, dev, rank, local_rank, world, peaks, full=False, ceiling=res["ceiling"])
            r.pop("leg")
            r.pop("ceiling")
            r["config"] = config_of(w2, args)["workload"]
            extra[name] = r

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    line = {
        "metric": METRIC, "value": res["value"], "unit": "TOPS", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "i8", "data": "synthetic", "config": config_of(wl, args),
        "roofline": res["roofline"], "roofline_rotate_quantize": res["roofline_rotate_quantize"],
        "int8_ceiling": res["ceiling"], "stages": res["stages"], "other_layout": res.get("other_layout"),
        "e2e": e2e, "gpu_launches": res["gpu_launches"], "clocks": res["clocks"],
    }
    if extra is not None:
        line["workloads"] = extra
    if not args.no_cpu_baseline and world == 1:
        dt, ops, threads = oracle_sample(wl, args.ref_tokens, scale_group=args.scale_group)
        line["cpu_baseline"] = {"value": ops / dt / 1e12, "unit": "TOPS", "cores": threads, "kind": "oracle",
                                "sample": f"{args.ref_tokens} tokens of each layer of '{wl.name}' (full K and N), {dt:.1f} s"}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def run_e2e(args, wl, leg, dev, B, dist, world):
    """Same metric through the user-facing call dvdq_qlinear, with the layer input copied from
    pinned host memory and the layer output copied back to pinned host memory inside every step.
    Three streams (copy-in, compute, copy-out) and two device input buffers let the PCIe copies of
    neighbouring layers overlap the kernels; every byte still crosses the bus inside the timed region.
    (In the chain workload every layer's input is copied in like the others': the host holds it.)"""
    M = wl.M
    layers = leg.layers
    maxK = max(L["layer"].K for L in layers)
    maxN = max(L["layer"].N for L in layers)
    host_x = {}
    for L in layers:
        if L["layer"].K not in host_x:
            host_x[L["layer"].K] = L["x"].to("cpu").pin_memory()
    host_y = [torch.empty(M, maxN, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    dev_x = [torch.empty(M, maxK, dtype=torch.bfloat16, device=dev) for _ in range(2)]
    # room for the int8 weight operand behind the codes: dvdq_qlinear then writes it once per call
    extra = 0 if args.weight_operand == "tile" else max(B.dvdq_weight_operand_bytes(L["layer"].N, L["layer"].K) for L in layers) + 256
    ws = torch.empty(max(B.dvdq_qlinear_workspace_bytes(M, L["layer"].K, L["q"]) for L in layers) + extra, dtype=torch.uint8, device=dev)
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
    ap.add_argument("--workload", default="hunyuan",
                    help="tiny, wan1p3b, hunyuan (default, the headline), wan14b, ffn_chain; 'all' = the headline plus a "
                         "'workloads' block with the per-layer figures of every other configuration")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--ref-tokens", type=int, default=384, help="token sample timed on the CPU oracle")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--tokens", type=int, default=0, help="override the workload's token count (profiling runs)")
    ap.add_argument("--container", type=int, default=0,
                    help="0 (default): activation codes packed b bits each, widened inside the GEMM; "
                         "8: one int8 per code, read by the GEMM as they are")
    ap.add_argument("--no-other-layout", "--no-packed", dest="no_other_layout", action="store_true",
                    help="skip the extra leg that times the other code layout")
    ap.add_argument("--no-alone", action="store_true", help="skip the extra leg that times rotate-quantize on its own")
    ap.add_argument("--no-ceiling", action="store_true", help="skip the int8 issue-loop ceiling (the roofline then falls back to 2 x bf16)")
    ap.add_argument("--scale-group", type=int, default=0,
                    help="0: one activation scale per token; 128, 256, 1024: one per token and group of that many channels")
    ap.add_argument("--fuse", action="store_true",
                    help="chain workloads: every layer but the last writes the next layer's codes from its epilogue "
                         "(dvdq_qgemm_fused_rq, rotation block = scale group = 256) instead of bf16; needs --container 8")
    ap.add_argument("--weight-operand", default="launch", choices=["launch", "tile", "resident"],
                    help="where the GEMM's int8 weight operand comes from: written into a scratch area by a widening "
                         "kernel before every GEMM launch, inside the timed region (launch); widened inside the GEMM by "
                         "every output tile (tile); or written once and kept, 8 more bits per weight (resident)")
    ap.add_argument("--bits", type=int, default=0, help="override the activation bit width of every layer (4, 6 or 8)")
    args = ap.parse_args()
    from paper_2505_18663_b200 import workloads as W
    args.all_workloads = args.workload == "all"
    wl = W.WORKLOADS["hunyuan" if args.all_workloads else args.workload]
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
