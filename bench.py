#!/usr/bin/env python
"""Benchmark of the fp4q hot path on B200.

One step = one pass of the whole path over one batch of seeded synthetic tensors of the 7B-class dense
layer configuration (hidden 4096, FFN 11008, 16384 tokens): the 2D-block FP4 quantize + dual-layout pack
of every operand (7 weights, 4 distinct activations, 7 output gradients, stochastic rounding) followed by
the forward, dgrad and wgrad block-scaled FP4 GEMMs of the 7 linear layers.  The headline value is the
quantize+dual-pack throughput in GB/s (3.001 algorithmic bytes per element); the GEMM TFLOP/s per product
are reported beside it, and the MXFP8 query/key projections and the grouped MoE expert layer are timed
separately under "extras".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line (rank 0).  With --impl reference the CPU oracle is timed instead, on a bounded
sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

BYTES_PER_ELEMENT = 2.0 + 0.5 + 0.5 + 1.0 / 1024.0   # BF16 read, two packed layouts, one scale byte per 32x32 block
METRIC = "2D-FP4 quantize+dual-pack GB/s; block-scaled FP4 GEMM TFLOPS (fwd/dgrad/wgrad)"
FP4_OVER_BF16 = 4.0      # nominal dense tensor-core ratio (9 PFLOP/s FP4 : 2.25 PFLOP/s BF16)
FP8_OVER_BF16 = 2.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs (reads only)."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: str):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(prefix="fp4q_clocks_", suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    @staticmethod
    def _stamp(text):
        import datetime
        try:
            return datetime.datetime.strptime(text, "%Y/%m/%d %H:%M:%S.%f").timestamp()
        except ValueError:
            return None

    def stop(self, window=None):
        """window = (t_start, t_end) in host time.time() seconds: only samples taken inside it count (when there
        are none - a very short region - all samples taken after t_start minus one period do)."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        try:
            with open(self.path) as f:
                for line in f:
                    t = [x.strip() for x in line.split(",")]
                    if len(t) < 9:
                        continue
                    try:
                        rows.append((self._stamp(t[0]), float(t[1]), float(t[2]), float(t[3]), t[5:9]))
                    except ValueError:
                        continue
            os.unlink(self.path)
        except Exception:
            pass
        if window is not None and rows:
            inside = [r for r in rows if r[0] is not None and window[0] <= r[0] <= window[1]]
            rows = inside or [r for r in rows if r[0] is not None and r[0] >= window[0] - 0.05] or rows
        if rows:
            reasons = set()
            for r in rows:
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            out.update(sm_mhz=statistics.median([r[1] for r in rows]), sm_max_mhz=max(r[2] for r in rows),
                       power_w=statistics.median([r[3] for r in rows]), reasons=sorted(reasons), samples=len(rows))
        return out


# ------------------------------------------------------------------------------------------ multi-rank

def max_over_ranks(values, dist, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (replicas are timed by the slowest one)."""
    if dist is None:
        return [float(v) for v in values]
    import torch
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.cpu().tolist()


def aggregate_throughput(units_per_rank, world, ms):
    """Whole-job throughput of `world` replicas that each processed units_per_rank in ms (max over ranks)."""
    return world * units_per_rank / (ms * 1e-3)


def launcher_command(n_ranks, argv, port=None):
    """The command that starts n_ranks copies of this script, one per GPU (torch.distributed.run on this node)."""
    port = port or (29500 + os.getpid() % 2000)
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n_ranks),
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def relaunch_as_ranks(args, argv):
    """`--gpus N` with N > 1 outside a torchrun launch: start the N ranks here and hand their exit code back."""
    return subprocess.call(launcher_command(args.gpus, argv))


def run_rank_selftest(args):
    """Host-side logic of the N > 1 path on CPU ranks (gloo): rendezvous, max over ranks, aggregation, one JSON line
    from rank 0.  Used by the tests; touches no GPU."""
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    ms = max_over_ranks([10.0 + rank], dist if world > 1 else None, "cpu")[0]
    if world > 1:
        dist.barrier()
    if rank == 0:
        print(json.dumps({"selftest": True, "n_gpus": world, "ms_per_step": ms,
                          "value": aggregate_throughput(1000.0, world, ms), "scaling": "weak"}))
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------ workload

def build_dense_workload(cfg, device, torch, workloads):
    """All BF16 operands of one dense layer set: per layer W [N,K], X [T,K] (shared between layers with the
    same input), dY [T,N]."""
    T = cfg.tokens
    layers = cfg.layers()
    x_of = {"q": "attn_in", "k": "attn_in", "v": "attn_in", "o": "o_in", "gate": "mlp_in", "up": "mlp_in", "down": "down_in"}
    xs, ops = {}, []
    for i, (name, n, k) in enumerate(layers):
        key = x_of[name]
        if key not in xs:
            xs[key] = workloads.activations_student_t(T, k, cfg.data_seed + 10 * i + 1, device, nu=cfg.nu)
        ops.append({"name": name, "N": n, "K": k, "W": workloads.weights(n, k, cfg.data_seed + 10 * i, device),
                    "X": xs[key], "x_key": key, "dY": workloads.gradients_rowscaled(T, n, cfg.data_seed + 10 * i + 2, device)})
    return ops, xs


def run_gpu(args):
    import torch
    from paper_2607_24953_b200 import binding, workloads

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit("bench.py: --gpus %d but the launch has %d rank(s)" % (args.gpus, world))
    if torch.cuda.device_count() < world:
        raise SystemExit("bench.py: %d ranks need %d GPUs, %d visible" % (world, world, torch.cuda.device_count()))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)
    binding.lib()   # fail loudly if the CUDA library is missing

    cfg = {"7b": workloads.CONFIG_7B, "1b": workloads.CONFIG_1B, "tiny": workloads.CONFIG_TINY}[args.workload]
    T = cfg.tokens
    ops, xs = build_dense_workload(cfg, dev, torch, workloads)
    seed = cfg.philox_seed
    SR = binding.ROUND_STOCHASTIC

    # quantize targets: 7 W, the distinct X, 7 dY -- preallocated outputs
    q_w = [binding.alloc_qtensor(o["N"], o["K"], dev) for o in ops]
    q_x = {k: binding.alloc_qtensor(T, v.shape[1], dev) for k, v in xs.items()}
    q_dy = [binding.alloc_qtensor(T, o["N"], dev) for o in ops]
    quant_jobs = [(o["W"], q_w[i], 10 * i) for i, o in enumerate(ops)]
    quant_jobs += [(xs[k], q_x[k], 100 + j) for j, k in enumerate(xs)]
    quant_jobs += [(o["dY"], q_dy[i], 10 * i + 2) for i, o in enumerate(ops)]
    quant_elems = sum(t.numel() for t, _, _ in quant_jobs)
    quant_bytes = quant_elems * BYTES_PER_ELEMENT

    max_n, max_k = max(o["N"] for o in ops), max(o["K"] for o in ops)
    y_buf = torch.empty((T, max_n), dtype=torch.bfloat16, device=dev)
    dx_buf = torch.empty((T, max_k), dtype=torch.bfloat16, device=dev)
    dw_buf = torch.empty((max(o["N"] * o["K"] for o in ops),), dtype=torch.float32, device=dev)
    ws = binding.alloc_workspace(dev)
    gemm_flops = sum(2.0 * T * o["N"] * o["K"] for o in ops)
    # algorithmic bytes of the 21 GEMM launches: both operands' payloads and scales read once, the output written once
    # (forward and dgrad in BF16, wgrad in FP32)
    pay = lambda r, c: r * c * (0.5 + 1.0 / 1024)
    gemm_alg_bytes = sum(pay(T, o["K"]) + pay(o["N"], o["K"]) + 2.0 * T * o["N"] +        # forward
                         pay(T, o["N"]) + pay(o["N"], o["K"]) + 2.0 * T * o["K"] +        # dgrad
                         pay(T, o["N"]) + pay(T, o["K"]) + 4.0 * o["N"] * o["K"] for o in ops)

    def outputs(o):
        return (y_buf[:, :o["N"]], dx_buf[:, :o["K"]], dw_buf[:o["N"] * o["K"]].view(o["N"], o["K"]))

    ev = lambda: torch.cuda.Event(enable_timing=True)

    def phase_quantize_per_tensor():
        for x, q, tid in quant_jobs:
            binding.fp4q_quantize2d(x, q, mode=SR, seed=seed, tensor_id=tid)

    def phase_quantize():
        # all 18 operands by one call of the library's multi-tensor entry point (chained launches in one stream)
        binding.fp4q_quantize2d_multi([x for x, _, _ in quant_jobs], [q for _, q, _ in quant_jobs], mode=SR, seed=seed,
                                      tensor_ids=[tid for _, _, tid in quant_jobs])

    def phase_fwd():
        for i, o in enumerate(ops):
            binding.fp4q_gemm_fwd(q_x[o["x_key"]], q_w[i], out=outputs(o)[0], dt=binding.OUT_BF16, ws=ws)

    def phase_dgrad():
        for i, o in enumerate(ops):
            binding.fp4q_gemm_dgrad(q_dy[i], q_w[i], out=outputs(o)[1], dt=binding.OUT_BF16, ws=ws)

    def phase_wgrad():
        for i, o in enumerate(ops):
            binding.fp4q_gemm_wgrad(q_dy[i], q_x[o["x_key"]], out=outputs(o)[2], dt=binding.OUT_F32, ws=ws)

    side = [torch.cuda.Stream(device=dev) for _ in range(2)]

    def phase_quantize_two_streams():
        # the 18 operands are independent of one another: their launches alternate between two streams, so that one
        # kernel's last wave overlaps the next one's first (used for the graph capture only)
        cur = torch.cuda.current_stream()
        for st in side:
            st.wait_stream(cur)
        for n, (x, q, tid) in enumerate(quant_jobs):
            binding.fp4q_quantize2d(x, q, mode=SR, seed=seed, tensor_id=tid, stream=side[n & 1])
        for st in side:
            cur.wait_stream(st)

    quantize_variant = "two-streams" if args.two_stream_quantize else "per-tensor" if args.per_tensor_quantize else "multi"
    phases = [phase_quantize_per_tensor if quantize_variant != "multi" else phase_quantize, phase_fwd, phase_dgrad, phase_wgrad]

    def step(marks=None):
        for i, ph in enumerate(phases):
            if marks: marks[i].record()
            ph()
        if marks: marks[4].record()

    launches_per_step = len(quant_jobs) + 3 * len(ops)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = str(local_rank)
    sampler = ClockSampler(gpu_id)
    sampler.start()   # nvidia-smi needs a moment to start: it runs through the warm-up, samples are selected by time
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    if binding.fp4q_workspace_status(ws) != 0:
        raise RuntimeError("a GEMM kernel reported a device-side timeout during warm-up")
    if not args.no_graphs:
        # The step's launches are short (8 us for a 4096 x 4096 weight) against the cost of issuing them one by one
        # from Python: each phase is captured once into a CUDA graph (same kernels, same arguments, same order) and
        # the timed steps replay the graphs.
        graphs = []
        if quantize_variant == "two-streams":
            phases[0] = phase_quantize_two_streams
        for ph in list(phases):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                ph()
            graphs.append(g)
        phases[:] = [g.replay for g in graphs]
        step()
        barrier()

    marks = [[ev() for _ in range(5)] for _ in range(args.steps)]
    barrier()
    t0, t1 = ev(), ev()
    wall0 = time.time()
    t0.record()
    for s in range(args.steps):
        step(marks[s])
    t1.record()
    barrier()
    wall1 = time.time()
    clocks = sampler.stop((wall0, wall1))
    total_ms = t0.elapsed_time(t1)
    status = binding.fp4q_workspace_status(ws)
    if status != 0:
        raise RuntimeError("a GEMM kernel reported a device-side timeout: status %d" % status)

    phase_ms = np.array([[m[i].elapsed_time(m[i + 1]) for i in range(4)] for m in marks])   # quant, fwd, dgrad, wgrad
    red = max_over_ranks([total_ms] + phase_ms.sum(0).tolist(), dist, dev)
    total_ms, phase_tot = red[0], np.array(red[1:])
    ms_per_step = total_ms / args.steps
    q_ms, f_ms, d_ms, w_ms = (phase_tot / args.steps).tolist()
    quant_gbs = aggregate_throughput(quant_bytes, world, q_ms) / 1e9
    tf = lambda ms: aggregate_throughput(gemm_flops, world, ms) / 1e12
    gemm_tflops = {"fwd": tf(f_ms), "dgrad": tf(d_ms), "wgrad": tf(w_ms),
                   "all": aggregate_throughput(3 * gemm_flops, world, f_ms + d_ms + w_ms) / 1e12}

    # ---- end to end: pinned host inputs -> device, quantize + GEMMs, results -> pinned host
    e2e = None
    if not args.no_e2e:
        host_in = []
        for x, _, _ in quant_jobs:
            h = torch.empty(x.shape, dtype=x.dtype, pin_memory=True)
            h.copy_(x)
            host_in.append(h)
        host_out = [[torch.empty(b.shape, dtype=b.dtype, pin_memory=True) for b in outputs(o)] for o in ops]
        h2d = sum(h.numel() * h.element_size() for h in host_in)
        d2h = sum(b.numel() * b.element_size() for bs in host_out for b in bs)

        # Three streams: host->device copies, the kernels, device->host copies.  PCIe carries both directions at once, so
        # the copies in are hidden behind the copies out; the kernels wait for their inputs' copy, an output buffer (shared
        # by the layers) is rewritten only after its previous contents have left, and an input buffer is refilled only
        # after the quantize kernel that read it.
        s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        cur = torch.cuda.current_stream()
        quant_done = [None]
        out_copied = [None, None, None]

        def e2e_step():
            if quant_done[0] is not None:
                s_in.wait_event(quant_done[0])
            for (x, q, tid), h in zip(quant_jobs, host_in):
                with torch.cuda.stream(s_in):
                    x.copy_(h, non_blocking=True)
                    arrived = torch.cuda.Event()
                    arrived.record(s_in)
                cur.wait_event(arrived)
                binding.fp4q_quantize2d(x, q, mode=SR, seed=seed, tensor_id=tid)
            quant_done[0] = torch.cuda.Event()
            quant_done[0].record(cur)
            for i, o in enumerate(ops):
                bufs = outputs(o)
                calls = (lambda: binding.fp4q_gemm_fwd(q_x[o["x_key"]], q_w[i], out=bufs[0], dt=binding.OUT_BF16, ws=ws),
                         lambda: binding.fp4q_gemm_dgrad(q_dy[i], q_w[i], out=bufs[1], dt=binding.OUT_BF16, ws=ws),
                         lambda: binding.fp4q_gemm_wgrad(q_dy[i], q_x[o["x_key"]], out=bufs[2], dt=binding.OUT_F32, ws=ws))
                for k in range(3):
                    if out_copied[k] is not None:
                        cur.wait_event(out_copied[k])
                    calls[k]()
                    produced = torch.cuda.Event()
                    produced.record(cur)
                    with torch.cuda.stream(s_out):
                        s_out.wait_event(produced)
                        host_out[i][k].copy_(bufs[k], non_blocking=True)
                        out_copied[k] = torch.cuda.Event()
                        out_copied[k].record(s_out)
            cur.wait_stream(s_out)   # the step ends when its last result is on the host

        e2e_steps = max(1, min(args.steps, 3))
        e2e_step()
        barrier()
        a, b = ev(), ev()
        a.record()
        for _ in range(e2e_steps):
            e2e_step()
        b.record()
        barrier()
        e_ms = a.elapsed_time(b) / e2e_steps
        e_ms = max_over_ranks([e_ms], dist, dev)[0]
        # same metric: quantize+dual-pack algorithmic bytes over the end-to-end step time
        e2e = {"value": aggregate_throughput(quant_bytes, world, e_ms) / 1e9, "unit": "GB/s", "ms_per_step": e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "note": "whole step (H2D of all BF16 operands, quantize sweep, 21 GEMMs, D2H of all outputs) with the "
                       "copies in, the kernels and the copies out on three streams; PCIe-bound"}
        del host_in, host_out

    # ---- per-operand quantize and GEMM rates (each launch timed on its own; a weight that fits in L2 is evicted first
    # by a write of a buffer larger than L2)
    per_operand = None
    if not args.no_extras and rank == 0:
        flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)

        def timed_cold(fn, iters=5):
            tot = 0.0
            for _ in range(iters + 1):
                flush.fill_(1)
                a, b = ev(), ev()
                a.record()
                fn()
                b.record()
                torch.cuda.synchronize()
                tot += a.elapsed_time(b)
                if _ == 0:
                    tot = 0.0      # first call: warm-up
            return tot / iters

        q_rates = {}
        names = ["W_" + o["name"] for o in ops] + ["X_" + k for k in xs] + ["dY_" + o["name"] for o in ops]
        for (x, q, tid), nm in zip(quant_jobs, names):
            ms = timed_cold(lambda: binding.fp4q_quantize2d(x, q, mode=SR, seed=seed, tensor_id=tid))
            q_rates[nm] = {"shape": list(x.shape), "gbs": x.numel() * BYTES_PER_ELEMENT / (ms * 1e-3) / 1e9}
        g_rates = {}
        for i, o in enumerate(ops):
            fl = 2.0 * T * o["N"] * o["K"]
            y, dx, dw = outputs(o)
            g_rates[o["name"]] = {
                "T_N_K": [T, o["N"], o["K"]],
                "fwd_tflops": fl / (timed_cold(lambda: binding.fp4q_gemm_fwd(q_x[o["x_key"]], q_w[i], out=y, ws=ws)) * 1e-3) / 1e12,
                "dgrad_tflops": fl / (timed_cold(lambda: binding.fp4q_gemm_dgrad(q_dy[i], q_w[i], out=dx, ws=ws)) * 1e-3) / 1e12,
                "wgrad_tflops": fl / (timed_cold(lambda: binding.fp4q_gemm_wgrad(q_dy[i], q_x[o["x_key"]], out=dw, dt=binding.OUT_F32, ws=ws)) * 1e-3) / 1e12}
        per_operand = {"quantize": q_rates, "gemm": g_rates,
                       "note": "one launch at a time, L2 flushed before each (256 MB written), mean of 5"}
        del flush

    extras = {}
    if not args.no_extras:
        extras = run_extras(torch, binding, workloads, dev, ws, measured_peaks())
        if per_operand is not None:
            extras["per_operand"] = per_operand

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    # The measured BF16 peak comes in two regimes: single launches at full clock ("burst") and a seconds-long loop
    # under the power cap ("sustained").  The timed region is compared with the regime its sampled clocks show.
    burst_regime = (clocks.get("sm_mhz") is not None and clocks.get("sm_max_mhz") and
                    clocks["sm_mhz"] >= 0.93 * clocks["sm_max_mhz"] and "sw_power_cap" not in clocks.get("reasons", []))
    regime = "burst" if burst_regime else "sustained"
    bf16_peak = peaks["bf16_tflops"] if burst_regime else peaks["bf16_tflops_sustained"]
    fp4_peak = bf16_peak * FP4_OVER_BF16
    gemm_ms_per_launch = (f_ms + d_ms + w_ms) / (3 * len(ops))
    achieved_tf = 3 * gemm_flops / ((f_ms + d_ms + w_ms) * 1e-3) / 1e12
    roofline = {"kernel": "gemm_block_scaled_kernel<mxf4>", "bound": "tensor", "achieved": achieved_tf, "peak": fp4_peak,
                "unit": "TFLOP/s", "frac": achieved_tf / fp4_peak, "traffic": None,
                "peak_source": "%s bf16 %s %.1f TFLOP/s x %.0f (nominal FP4:BF16 ratio); clocks in the timed region "
                               "match the %s regime" % (peaks["source"], regime, bf16_peak, FP4_OVER_BF16, regime),
                "frac_of_burst_peak": achieved_tf / (peaks["bf16_tflops"] * FP4_OVER_BF16),
                "frac_of_sustained_peak": achieved_tf / (peaks["bf16_tflops_sustained"] * FP4_OVER_BF16),
                "frac_of_nominal_9pf": achieved_tf / 9000.0,
                "flops_per_launch": 3 * gemm_flops / (3 * len(ops)), "ms_per_launch": gemm_ms_per_launch,
                "algorithmic_bytes_per_launch": gemm_alg_bytes / (3 * len(ops)),
                "time_share_of_step": (f_ms + d_ms + w_ms) / ms_per_step}
    q_gbs_1 = quant_bytes / (q_ms * 1e-3) / 1e9
    roofline_quantize = {"kernel": "quantize2d_kernel<stochastic>", "bound": "hbm", "achieved": q_gbs_1,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": q_gbs_1 / peaks["hbm_gbs"], "traffic": None,
                         "peak_source": peaks["source"] + " copy bandwidth",
                         "bytes_per_launch": quant_bytes / len(quant_jobs), "ms_per_launch": q_ms / len(quant_jobs),
                         "time_share_of_step": q_ms / ms_per_step}
    if not args.no_graphs:
        # the sweep on its own (no GEMMs between repetitions, so at cooler clocks than inside the step): the library's
        # multi-tensor call, one plain launch per tensor in one stream, and plain launches alternating between two streams
        def captured(fn):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn()
            return g

        def sweep_rate(replay):
            replay()
            torch.cuda.synchronize()
            a, b = ev(), ev()
            a.record()
            for _ in range(10):
                replay()
            b.record()
            torch.cuda.synchronize()
            return quant_bytes / (a.elapsed_time(b) / 10 * 1e-3) / 1e9

        roofline_quantize["sweep_alone_gbs"] = {"multi_tensor_call": sweep_rate(captured(phase_quantize).replay),
                                                "per_tensor_one_stream": sweep_rate(captured(phase_quantize_per_tensor).replay),
                                                "per_tensor_two_streams": sweep_rate(captured(phase_quantize_two_streams).replay)}
        roofline_quantize["note"] = ("the timed step quantizes its 18 operands with the '%s' variant; sweep_alone_gbs compares "
                                     "the three variants of the sweep run on their own; launches of independent operands overlap, "
                                     "so ms_per_launch is the phase time divided by the launch count" % quantize_variant)
    fill_traffic(roofline, roofline_quantize)

    cpu = cpu_baseline_quantize(workloads, cfg, seconds=args.cpu_seconds)
    inputs_sha256 = None
    if not args.no_hash:
        import hashlib
        names = ["W_" + o["name"] for o in ops] + ["X_" + k for k in xs] + ["dY_" + o["name"] for o in ops]
        digest_all, per = hashlib.sha256(), {}
        for (x, _, _), nm in zip(quant_jobs, names):
            h = hashlib.sha256(workloads.bf16_bits(x).tobytes()).hexdigest()
            per[nm] = h[:16]
            digest_all.update(bytes.fromhex(h))
        inputs_sha256 = {"all": digest_all.hexdigest(), "per_tensor_first16": per,
                         "note": "SHA-256 of each BF16 operand's bytes (row-major); 'all' hashes the 18 digests in sweep order"}

    line = {
        "metric": METRIC, "value": quant_gbs, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "fp4-e2m1 (bf16 in, fp32 accumulate)", "data": "synthetic",
        "config": {"workload": cfg.name + ": hidden %d, FFN %d, %d tokens; quantize sweep over 7 W + %d X + 7 dY "
                               "(stochastic rounding) then fwd/dgrad/wgrad FP4 GEMMs of 7 linear layers" %
                               (cfg.hidden, cfg.ffn, cfg.tokens, len(xs)),
                   "parallelism": "replicas only (x%d)" % world,
                   "launch": "per-launch calls from Python" if args.no_graphs else
                             "one CUDA graph per phase (quantize, fwd, dgrad, wgrad), replayed" +
                             {"multi": "; the quantize sweep is one fp4q_quantize2d_multi call (18 chained launches in one stream)",
                              "per-tensor": "; one plain quantize launch per tensor",
                              "two-streams": "; the quantize sweep's per-tensor launches alternate between two streams"}[quantize_variant], "l2": "inputs larger than L2 (%.2f GB of BF16 operands per step)" %
                   (quant_elems * 2 / 1e9), "quantize_bytes_per_step": quant_bytes, "gemm_flops_per_step": 3 * gemm_flops},
        "gemm_tflops": gemm_tflops,
        "phase_ms": {"quantize": q_ms, "fwd": f_ms, "dgrad": d_ms, "wgrad": w_ms},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
        "roofline": roofline, "roofline_quantize": roofline_quantize, "cpu_baseline": cpu, "inputs_sha256": inputs_sha256,
        "extras": extras,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def fill_traffic(roofline, roofline_quantize):
    """DRAM traffic per launch from the committed ncu summaries (profiles/traffic.json), if present."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return
    try:
        with open(path) as f:
            t = json.load(f)
        # captured on a smaller case and scaled by the units processed (traffic grows in proportion)
        if "gemm_dram_over_algorithmic" in t:   # measured on one full-size launch (7B gate/up shape)
            roofline["traffic"] = t["gemm_dram_over_algorithmic"] * roofline["algorithmic_bytes_per_launch"]
        if "quantize_dram_bytes_per_algorithmic_byte" in t:
            roofline_quantize["traffic"] = t["quantize_dram_bytes_per_algorithmic_byte"] * roofline_quantize["bytes_per_launch"]
    except Exception:
        pass


def bound_of(flops, alg_bytes, tensor_tflops, hbm_gbs):
    """Roofline of one product: the slower of its flops at the tensor peak and its algorithmic bytes at the HBM rate."""
    t_tensor, t_hbm = flops / (tensor_tflops * 1e12), alg_bytes / (hbm_gbs * 1e9)
    return {"bound": "tensor" if t_tensor >= t_hbm else "hbm", "ms": max(t_tensor, t_hbm) * 1e3}


def run_extras(torch, binding, workloads, dev, ws, peaks):
    """MXFP8 query/key projections at 7B shapes and the grouped MoE expert layer, timed on their own."""
    out = {}
    fp4_peak, fp8_peak, hbm = peaks["bf16_tflops"] * FP4_OVER_BF16, peaks["bf16_tflops"] * FP8_OVER_BF16, peaks["hbm_gbs"]
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def timed(fn, iters=5):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = ev(), ev()
        a.record()
        for _ in range(iters):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / iters

    # --- MXFP8 Q/K projections: X 16384x4096, Wq, Wk 4096x4096
    cfg = workloads.CONFIG_ATTN_7B
    T, H = cfg.tokens, cfg.hidden
    X = workloads.activations_student_t(T, H, cfg.data_seed + 1, dev, nu=cfg.nu)
    Wq, Wk = workloads.weights(H, H, cfg.data_seed, dev), workloads.weights(H, H, cfg.data_seed + 10, dev)
    xq, xs = binding.fp4q_mxfp8_quantize1d(X)
    wqq, wqs = binding.fp4q_mxfp8_quantize1d(Wq)
    wkq, wks = binding.fp4q_mxfp8_quantize1d(Wk)
    ms_q = timed(lambda: binding.fp4q_mxfp8_quantize1d(X))
    ms_g = timed(lambda: binding.fp4q_mxfp8_qk(xq, xs, wqq, wqs, wkq, wks, T, H, H, ws=ws))
    qk_tf = 2 * 2.0 * T * H * H / (ms_g * 1e-3) / 1e12
    out["mxfp8_qk"] = {"workload": "Q and K projections, %d tokens, %dx%d each" % (T, H, H),
                       "quantize_gbs": T * H * (3.0 + 1 / 32) / (ms_q * 1e-3) / 1e9,
                       "gemm_tflops": qk_tf, "gemm_ms": ms_g,
                       "roofline": {"kernel": "gemm_block_scaled_kernel<mxf8f6f4>", "bound": "tensor", "achieved": qk_tf, "peak": fp8_peak,
                                    "unit": "TFLOP/s", "frac": qk_tf / fp8_peak, "frac_of_nominal_4500": qk_tf / 4500.0,
                                    "peak_source": "%s bf16 burst %.1f TFLOP/s x %.0f (nominal FP8:BF16 ratio)" %
                                                   (peaks["source"], peaks["bf16_tflops"], FP8_OVER_BF16)}}
    # backward of the same projections: operands re-quantized along the new contraction axis
    dYq = workloads.gradients_rowscaled(T, H, cfg.data_seed + 2, dev)
    ms_qt = timed(lambda: binding.fp4q_mxfp8_quantize1d_t(X))
    dyq, dys = binding.fp4q_mxfp8_quantize1d(dYq)
    wtq, wts = binding.fp4q_mxfp8_quantize1d_t(Wq)
    dytq, dyts = binding.fp4q_mxfp8_quantize1d_t(dYq)
    xtq, xts = binding.fp4q_mxfp8_quantize1d_t(X)
    ms_dg = timed(lambda: binding.fp4q_mxfp8_gemm(dyq, dys, wtq, wts, T, H, H, ws=ws))
    ms_wg = timed(lambda: binding.fp4q_mxfp8_gemm(dytq, dyts, xtq, xts, H, H, T, dt=binding.OUT_F32, ws=ws))
    out["mxfp8_backward"] = {"workload": "dX = dY Wq and dWq = dY^T X of one projection, %d tokens, %dx%d" % (T, H, H),
                             "transposing_quantize_gbs": T * H * (3.0 + 1 / 32) / (ms_qt * 1e-3) / 1e9,
                             "dgrad_tflops": 2.0 * T * H * H / (ms_dg * 1e-3) / 1e12,
                             "wgrad_tflops": 2.0 * T * H * H / (ms_wg * 1e-3) / 1e12}
    del xq, xs, wqq, wqs, wkq, wks, dYq, dyq, dys, wtq, wts, dytq, dyts, xtq, xts

    # --- forward product with the output quantization fused into the epilogue, against product + separate quantize
    qx4, qw4 = binding.fp4q_quantize2d(X), binding.fp4q_quantize2d(Wq)
    y = torch.empty(T, H, dtype=torch.bfloat16, device=dev)
    qy = binding.alloc_qtensor(T, H, dev)
    SR = binding.ROUND_STOCHASTIC
    ms_f = timed(lambda: binding.fp4q_gemm_fwd_quantized(qx4, qw4, out=qy, mode=SR, seed=1, tensor_id=2, ws=ws))
    ms_p = timed(lambda: binding.fp4q_gemm_fwd(qx4, qw4, out=y, ws=ws))
    ms_s = timed(lambda: binding.fp4q_quantize2d(y, out=qy, mode=SR, seed=1, tensor_id=2))
    out["fused_epilogue_quantization"] = {
        "workload": "Y = X W^T, %d x %d x %d, output as 2D-block FP4 (stochastic rounding)" % (T, H, H),
        "fused_ms": ms_f, "product_ms": ms_p, "separate_quantize_ms": ms_s,
        "fused_tflops": 2.0 * T * H * H / (ms_f * 1e-3) / 1e12, "speedup_vs_unfused": (ms_p + ms_s) / ms_f}
    # --- block-size study (Table 4): quantize and forward product at block edges 16 / 32 / 64 on the same tensors
    bs = {}
    y32 = torch.empty(T, H, dtype=torch.bfloat16, device=dev)
    for b, flag in ((16, binding.BLOCK_16), (32, 0), (64, binding.BLOCK_64)):
        qxb, qwb = binding.fp4q_quantize2d(X, flags=flag), binding.fp4q_quantize2d(Wq, flags=flag)
        ms_qb = timed(lambda: binding.fp4q_quantize2d(X, out=qxb, mode=SR, seed=1, tensor_id=2, flags=flag))
        gemm = binding.fp4q_gemm_fwd_b16 if b == 16 else binding.fp4q_gemm_fwd
        ms_gb = timed(lambda: gemm(qxb, qwb, out=y32, ws=ws))
        bs[str(b)] = {"quantize_gbs": T * H * (3.0 + 1.0 / (b * b if b != 64 else 1024)) / (ms_qb * 1e-3) / 1e9,
                      "fwd_tflops": 2.0 * T * H * H / (ms_gb * 1e-3) / 1e12, "fwd_ms": ms_gb}
        del qxb, qwb
    for b in bs:
        bs[b]["fwd_relative_to_32"] = bs["32"]["fwd_ms"] / bs[b]["fwd_ms"]
    bs["paper_table4_relative_throughput"] = {"8": 0.85, "16": 0.92, "32": 1.0, "64": 1.05,
                                              "note": "the paper's idealised trend column, for context (block edge 8 is not built)"}
    out["block_sizes"] = {"workload": "X %d x %d, W %d x %d, forward product" % (T, H, H, H), **bs}
    del y32
    # --- the paper's mixed layout: activations in 1D blocks (two encodings of X), weights and gradients in 2D blocks
    dY4 = binding.fp4q_quantize2d(workloads.gradients_rowscaled(T, H, cfg.data_seed + 2, dev), mode=SR, seed=1, tensor_id=3)
    x1q, x1s = binding.fp4q_quantize1d(X)
    x1tq, x1ts = binding.fp4q_quantize1d_t(X)
    dw = torch.empty(H, H, dtype=torch.float32, device=dev)
    ms_q1 = timed(lambda: binding.fp4q_quantize1d(X))
    ms_q1t = timed(lambda: binding.fp4q_quantize1d_t(X))
    ms_f1 = timed(lambda: binding.fp4q_gemm_fwd_act1d(x1q, x1s, T, qw4, out=y, ws=ws))
    ms_w1 = timed(lambda: binding.fp4q_gemm_wgrad_act1d(dY4, x1tq, x1ts, H, out=dw, ws=ws))
    ms_w2 = timed(lambda: binding.fp4q_gemm_wgrad(dY4, qx4, out=dw, ws=ws))
    out["mixed_layout_1d_activations"] = {
        "workload": "X %d x %d in 1 x 32 blocks (row-wise for the forward product, transposed for the weight gradient), "
                    "W and dY %d x %d in 32 x 32 blocks" % (T, H, H, H),
        "quantize1d_gbs": T * H * (2.5 + 1 / 32) / (ms_q1 * 1e-3) / 1e9,
        "quantize1d_t_gbs": T * H * (2.5 + 1 / 32) / (ms_q1t * 1e-3) / 1e9,
        "fwd_tflops": 2.0 * T * H * H / (ms_f1 * 1e-3) / 1e12, "wgrad_tflops": 2.0 * T * H * H / (ms_w1 * 1e-3) / 1e12,
        "all_2d_fwd_tflops": 2.0 * T * H * H / (ms_p * 1e-3) / 1e12, "all_2d_wgrad_tflops": 2.0 * T * H * H / (ms_w2 * 1e-3) / 1e12}
    del X, Wq, Wk, qx4, qw4, y, qy, dY4, x1q, x1s, x1tq, x1ts, dw

    # --- grouped MoE expert layer: 128 experts, hidden 2048, expert FFN 768, top-8 of 16384 tokens; token groups padded
    # to 128 rows (the configuration's figure) and to 256 rows, which lets forward and input gradient run on CTA pairs
    moe = workloads.CONFIG_MOE
    counts = workloads.moe_routing(moe)
    for pad, key in ((moe.pad, "moe_grouped"), (256, "moe_grouped_groups_padded_to_256")):
        offs = workloads.padded_row_offsets(counts, pad)
        Tp = int(offs[-1])
        d_offs = torch.from_numpy(offs).to(dev)
        E, H, F = moe.experts, moe.hidden, moe.expert_ffn
        res = {"workload": "%d experts, hidden %d, expert FFN %d, %d routed rows padded to %d; loads max %d / median %d / min %d" %
                           (E, H, F, int(counts.sum()), Tp, int(counts.max()), int(np.median(counts)), int(counts.min()))}
        tot_ms, tot_flops = 0.0, 0.0
        for name, n, k in moe.layers():
            Xm = workloads.zero_padding_rows(workloads.activations_student_t(Tp, k, moe.data_seed + 1, dev), counts, offs)
            dYm = workloads.zero_padding_rows(workloads.gradients_rowscaled(Tp, n, moe.data_seed + 2, dev), counts, offs)
            Wm = workloads.weights(E * n, k, moe.data_seed, dev)
            qx, qw, qdy = (binding.fp4q_quantize2d(t, mode=1, seed=moe.philox_seed, tensor_id=i) for i, t in enumerate((Xm, Wm, dYm)))
            y = torch.empty((Tp, n), dtype=torch.bfloat16, device=dev)
            dx = torch.empty((Tp, k), dtype=torch.bfloat16, device=dev)
            dw = torch.empty((E * n, k), dtype=torch.float32, device=dev)
            flops = 2.0 * float(counts.sum()) * n * k      # routed rows only: padding rows are not counted as work
            ms = [timed(lambda: binding.fp4q_gemm_fwd(qx, qw, out=y, row_offsets=d_offs, ws=ws, row_alignment=pad)),
                  timed(lambda: binding.fp4q_gemm_dgrad(qdy, qw, out=dx, row_offsets=d_offs, ws=ws, row_alignment=pad)),
                  timed(lambda: binding.fp4q_gemm_wgrad(qdy, qx, out=dw, row_offsets=d_offs, ws=ws))]
            # each product against its own bound: operand payloads + scales read once, output written once
            pay = lambda r, c: r * c * (0.5 + 1.0 / 1024)
            alg = [pay(Tp, k) + pay(E * n, k) + Tp * n * 2.0, pay(Tp, n) + pay(E * n, k) + Tp * k * 2.0,
                   pay(Tp, n) + pay(Tp, k) + E * n * k * 4.0]
            bounds = [bound_of(flops, a, fp4_peak, hbm) for a in alg]
            res[name] = {"fwd_tflops": flops / (ms[0] * 1e-3) / 1e12, "dgrad_tflops": flops / (ms[1] * 1e-3) / 1e12,
                         "wgrad_tflops": flops / (ms[2] * 1e-3) / 1e12, "ms": ms,
                         "wgrad_output_gbs": E * n * k * 4 / (ms[2] * 1e-3) / 1e9,
                         "bound": {nm: {"kind": b["bound"], "bound_ms": b["ms"], "frac": b["ms"] / m}
                                   for nm, b, m in zip(("fwd", "dgrad", "wgrad"), bounds, ms)}}
            if pad == 256:   # forward product with the output quantization in the epilogue, against product + quantize
                qy = binding.alloc_qtensor(Tp, n, dev)
                ms_fq = timed(lambda: binding.fp4q_gemm_fwd_quantized(qx, qw, out=qy, mode=1, seed=1, tensor_id=9, ws=ws, row_offsets=d_offs))
                ms_q = timed(lambda: binding.fp4q_quantize2d(y, out=qy, mode=1, seed=1, tensor_id=9))
                res[name]["fwd_quantized_ms"] = ms_fq
                res[name]["fwd_quantized_speedup_vs_unfused"] = (ms[0] + ms_q) / ms_fq
                del qy
            tot_ms += sum(ms)
            tot_flops += 3 * flops
            del Xm, dYm, Wm, qx, qw, qdy, y, dx, dw
        res["all_tflops"] = tot_flops / (tot_ms * 1e-3) / 1e12
        res["bound_note"] = ("per product: bound_ms = max(flops / (measured BF16 burst x 4), algorithmic bytes / measured copy "
                             "bandwidth); frac = bound_ms / measured ms")
        out[key] = res
    if binding.fp4q_workspace_status(ws) != 0:
        out["status"] = "device-side timeout reported"
    return out


# ------------------------------------------------------------------------------------------ CPU oracle legs

def cpu_baseline_quantize(workloads, cfg, seconds=12.0):
    """The oracle quantizer, as it stands, timed on the host cores on a bounded row slab of the largest
    activation (stochastic rounding, same seed)."""
    import oracle
    cols = cfg.ffn
    probe_rows = 64
    x = workloads.bf16_bits(workloads.activations_student_t(probe_rows, cols, cfg.data_seed + 61, "cpu", nu=cfg.nu))
    t0 = time.perf_counter()
    oracle.quantize2d(x, oracle.MODE_STOCHASTIC, seed=cfg.philox_seed, tensor_id=7)
    dt = max(time.perf_counter() - t0, 1e-6)
    rows = int(min(cfg.tokens, max(probe_rows, (seconds / dt) * probe_rows // 32 * 32)))
    x = workloads.bf16_bits(workloads.activations_student_t(rows, cols, cfg.data_seed + 61, "cpu", nu=cfg.nu))
    t0 = time.perf_counter()
    oracle.quantize2d(x, oracle.MODE_STOCHASTIC, seed=cfg.philox_seed, tensor_id=7)
    dt = time.perf_counter() - t0
    # the GEMM oracle (dequantize + float64 matmul) on a row sample of the largest forward product
    g_rows = 256
    xs = x[:g_rows]
    wbits = workloads.bf16_bits(workloads.weights(512, cols, cfg.data_seed + 60, "cpu"))
    qx, qw = oracle.quantize2d(xs, oracle.MODE_NEAREST), oracle.quantize2d(wbits, oracle.MODE_NEAREST)
    t1 = time.perf_counter()
    xd = oracle.dequantize2d(qx[0], qx[2], g_rows, cols)
    wd = oracle.dequantize2d(qw[0], qw[2], 512, cols)
    oracle.gemm_fwd(xd, wd)
    g_dt = max(time.perf_counter() - t1, 1e-9)
    # the tiny linear layer (W 256x256, X and dY 128x256) in full: three quantizations and the three products
    tiny = {k: workloads.bf16_bits(v) for k, v in workloads.tiny_layer("cpu").items()}
    t2 = time.perf_counter()
    tq = {k: oracle.quantize2d(v, oracle.MODE_STOCHASTIC, seed=0, tensor_id=i) for i, (k, v) in enumerate(tiny.items())}
    t3 = time.perf_counter()
    td = {k: oracle.dequantize2d(q[0], q[2], tiny[k].shape[0], tiny[k].shape[1]) for k, q in tq.items()}
    oracle.gemm_fwd(td["X"], td["W"]); oracle.gemm_dgrad(td["dY"], td["W"]); oracle.gemm_wgrad(td["dY"], td["X"])
    t4 = time.perf_counter()
    tiny_elems = sum(v.size for v in tiny.values())
    tiny_full = {"quantize_gbs": tiny_elems * BYTES_PER_ELEMENT / max(t3 - t2, 1e-9) / 1e9,
                 "gemm_gflops": 3 * 2.0 * 128 * 256 * 256 / max(t4 - t3, 1e-9) / 1e9,
                 "sample": "the tiny linear layer in full: 3 quantizations, then dequantize + the 3 float64 products"}
    return {"value": rows * cols * BYTES_PER_ELEMENT / dt / 1e9, "unit": "GB/s", "cores": oracle.num_threads(),
            "kind": "oracle", "seconds": dt, "tiny_layer_full": tiny_full,
            "gemm": {"value": 2.0 * g_rows * 512 * cols / g_dt / 1e9, "unit": "GFLOP/s",
                     "sample": "forward product oracle (dequantize + float64 matmul) on %d x 512 x %d" % (g_rows, cols)},
            "sample": "quantize+dual-pack (stochastic) of a %dx%d row slab of the %dx%d down-projection activation" %
                      (rows, cols, cfg.tokens, cols)}


def run_reference(args):
    """--impl reference: the CPU oracle timed on the host cores; each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2607_24953_b200 import workloads
    cfg = {"7b": workloads.CONFIG_7B, "1b": workloads.CONFIG_1B, "tiny": workloads.CONFIG_TINY}[args.workload]
    rows = 256
    tensors = [workloads.bf16_bits(workloads.weights(rows, cfg.hidden, cfg.data_seed, "cpu")),
               workloads.bf16_bits(workloads.activations_student_t(rows, cfg.ffn, cfg.data_seed + 61, "cpu", nu=cfg.nu)),
               workloads.bf16_bits(workloads.gradients_rowscaled(rows, cfg.hidden, cfg.data_seed + 2, "cpu"))]
    elems = sum(t.size for t in tensors)
    n_tok, n_out, k = 32, 512, cfg.hidden

    def step():
        """Returns (seconds in the quantizer, seconds in dequantize + the three products)."""
        t0 = time.perf_counter()
        qs = [oracle.quantize2d(t, oracle.MODE_STOCHASTIC, seed=cfg.philox_seed, tensor_id=i) for i, t in enumerate(tensors)]
        t1 = time.perf_counter()
        wd = oracle.dequantize2d(qs[0][0], qs[0][2], rows, cfg.hidden)
        xd = oracle.dequantize2d(qs[2][0], qs[2][2], rows, cfg.hidden)
        oracle.gemm_fwd(xd[:n_tok], wd[:n_out])
        oracle.gemm_dgrad(xd[:n_tok, :rows], wd)
        oracle.gemm_wgrad(xd[:n_tok, :rows], xd[:n_tok])
        return t1 - t0, time.perf_counter() - t1

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    quant_s = gemm_s = 0.0
    for _ in range(args.steps):
        q_s, g_s = step()
        quant_s += q_s
        gemm_s += g_s
    total = time.perf_counter() - t0
    value = args.steps * elems * BYTES_PER_ELEMENT / quant_s / 1e9
    gemm_flops = 2.0 * n_tok * (n_out * k + rows * cfg.hidden + rows * cfg.hidden)
    sample = ("per step: oracle quantize+dual-pack (stochastic) of %d-row slabs of a weight, the down-projection "
              "activation and an output gradient (%d elements), then the three float64 products on %d sampled rows" %
              (rows, elems, n_tok))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": total / args.steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name + " (bounded sample)", "parallelism": "host cores"},
            "gemm_tflops": {"all": args.steps * gemm_flops / max(gemm_s, 1e-9) / 1e12},
            "cpu_baseline": {"value": value, "unit": "GB/s", "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_kernel(args):
    """--kernel: one kernel on one shape, a few launches, for ncu captures and quick checks (one JSON line)."""
    import torch
    from paper_2607_24953_b200 import binding, workloads
    dev = torch.device("cuda", 0)
    dims = [int(v) for v in args.shape.lower().split("x")]
    ev = lambda: torch.cuda.Event(enable_timing=True)
    if args.kernel == "quantize":
        rows, cols = dims
        x = workloads.activations_student_t(rows, cols, 1, dev)
        out = binding.alloc_qtensor(rows, cols, dev)
        fn = lambda: binding.fp4q_quantize2d(x, out, mode=args.mode, seed=3, tensor_id=1)
        units, unit = rows * cols * BYTES_PER_ELEMENT / 1e9, "GB/s"
    elif args.kernel in ("quantize1d", "quantize1d_t"):
        rows, cols = dims
        x = workloads.activations_student_t(rows, cols, 1, dev)
        fn = (lambda: binding.fp4q_quantize1d(x)) if args.kernel == "quantize1d" else (lambda: binding.fp4q_quantize1d_t(x))
        units, unit = rows * cols * (2.5 + 1 / 32) / 1e9, "GB/s"
    elif args.kernel in ("gemm_fwd_act1d", "gemm_wgrad_act1d", "mxfp8_gemm"):
        T, N, K = dims
        ws = binding.alloc_workspace(dev)
        x = workloads.activations_student_t(T, K, 1, dev)
        if args.kernel == "gemm_fwd_act1d":
            xq, xs = binding.fp4q_quantize1d(x)
            qw = binding.fp4q_quantize2d(workloads.weights(N, K, 2, dev))
            out = torch.empty((T, N), dtype=torch.bfloat16, device=dev)
            fn = lambda: binding.fp4q_gemm_fwd_act1d(xq, xs, T, qw, out=out, ws=ws)
        elif args.kernel == "gemm_wgrad_act1d":
            xtq, xts = binding.fp4q_quantize1d_t(x)
            qdy = binding.fp4q_quantize2d(workloads.gradients_rowscaled(T, N, 3, dev), mode=1, seed=3, tensor_id=2)
            out = torch.empty((N, K), dtype=torch.float32, device=dev)
            fn = lambda: binding.fp4q_gemm_wgrad_act1d(qdy, xtq, xts, K, out=out, ws=ws)
        else:
            xq, xs = binding.fp4q_mxfp8_quantize1d(x)
            wq, wsf = binding.fp4q_mxfp8_quantize1d(workloads.weights(N, K, 2, dev))
            fn = lambda: binding.fp4q_mxfp8_gemm(xq, xs, wq, wsf, T, N, K, ws=ws)
        units, unit = 2.0 * T * N * K / 1e12, "TFLOP/s"
    else:
        T, N, K = dims
        ws = binding.alloc_workspace(dev)
        qx = binding.fp4q_quantize2d(workloads.activations_student_t(T, K, 1, dev), mode=1, seed=3, tensor_id=1)
        qw = binding.fp4q_quantize2d(workloads.weights(N, K, 2, dev), mode=1, seed=3, tensor_id=0)
        qdy = binding.fp4q_quantize2d(workloads.gradients_rowscaled(T, N, 3, dev), mode=1, seed=3, tensor_id=2)
        if args.kernel == "gemm_fwd_b16":
            qx16 = binding.fp4q_quantize2d(workloads.activations_student_t(T, K, 1, dev), flags=binding.BLOCK_16)
            qw16 = binding.fp4q_quantize2d(workloads.weights(N, K, 2, dev), flags=binding.BLOCK_16)
            out = torch.empty((T, N), dtype=torch.bfloat16, device=dev)
            fn = lambda: binding.fp4q_gemm_fwd_b16(qx16, qw16, out=out, ws=ws)
        elif args.kernel == "gemm_fwd":
            out = torch.empty((T, N), dtype=torch.bfloat16, device=dev)
            fn = lambda: binding.fp4q_gemm_fwd(qx, qw, out=out, ws=ws)
        elif args.kernel == "gemm_dgrad":
            out = torch.empty((T, K), dtype=torch.bfloat16, device=dev)
            fn = lambda: binding.fp4q_gemm_dgrad(qdy, qw, out=out, ws=ws)
        else:
            out = torch.empty((N, K), dtype=torch.float32, device=dev)
            fn = lambda: binding.fp4q_gemm_wgrad(qdy, qx, out=out, ws=ws)
        units, unit = 2.0 * T * N * K / 1e12, "TFLOP/s"
    fn()
    torch.cuda.synchronize()
    a, b = ev(), ev()
    a.record()
    for _ in range(args.iters):
        fn()
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / args.iters
    print(json.dumps({"kernel": args.kernel, "shape": args.shape, "iters": args.iters, "ms": ms,
                      "value": units / (ms * 1e-3), "unit": unit}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="fp4q", choices=["fp4q", "reference"])
    ap.add_argument("--workload", default="7b", choices=["7b", "1b", "tiny"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true")
    ap.add_argument("--no-hash", action="store_true", help="skip the SHA-256 of the input buffers")
    ap.add_argument("--no-graphs", action="store_true", help="issue every launch from Python instead of replaying CUDA graphs")
    ap.add_argument("--per-tensor-quantize", action="store_true", help="one fp4q_quantize2d launch per operand instead of the multi-tensor launch")
    ap.add_argument("--two-stream-quantize", action="store_true", help="per-operand launches alternating between two streams inside the graph")
    ap.add_argument("--rank-selftest", action="store_true", help=argparse.SUPPRESS)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--kernel", default=None, choices=["quantize", "gemm_fwd", "gemm_dgrad", "gemm_wgrad", "quantize1d", "quantize1d_t",
                                                        "gemm_fwd_act1d", "gemm_wgrad_act1d", "mxfp8_gemm", "gemm_fwd_b16"],
                    help="run one kernel on --shape a few times (for profiler captures) instead of the benchmark")
    ap.add_argument("--shape", default="16384x4096", help="RxC for quantize, TxNxK for the GEMMs")
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--mode", type=int, default=1, help="quantize rounding mode: 0 nearest, 1 stochastic")
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be at least 1")
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.kernel:
        # not under torchrun: start one rank per GPU (replicas; rank 0 prints the line with n_gpus = N)
        raise SystemExit(relaunch_as_ranks(args, sys.argv[1:]))
    if args.rank_selftest:
        run_rank_selftest(args)
    elif args.kernel:
        run_kernel(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
