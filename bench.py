#!/usr/bin/env python
"""Benchmark of the RMSMP layer path on B200.

Workload: the 19 3x3/1x1 convolutions of ResNet-18 at 224x224 input, batch 256 per GPU, run
layer by layer; every layer has its own seeded Kaiming weights (rows assigned PoT-4 : Fixed-4 :
Fixed-8 = 60:35:5 by variance rank) and its own seeded half-normal fp32 NHWC input.  One step is
one pass of the whole path over that batch: for every layer quantize+pack the fp32 weights,
quantize the fp32 activations to 4-bit codes, run the mixed-scheme implicit-GEMM convolution
(int32 accumulate, per-row scaled fp32 output).  Operations are counted as 2 per multiply-
accumulate (the convention of the paper's Table 6).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2111_00153_b200 import synth  # noqa: E402

METRIC = "mixed_scheme_gemm_tops"
UNIT = "TOPS"
RATIO = synth.RATIO_RMSMP1
BATCH = 256
WORKLOAD = "resnet18_conv_stack_3x3_1x1_224px_batch256_ratio60:35:5"


LAYER_FILTER = None    # set by --layers: comma-separated layer names, one instance each


def layer_list():
    out = []
    for L in synth.resnet18_convs():
        if LAYER_FILTER is not None:
            if L.name in LAYER_FILTER:
                out.append(L)
            continue
        for _ in range(L.count):
            out.append(L)
    return out


def host_layer(idx, L, batch, rank=0):
    """Weights are seeded by layer only (every rank holds the same, replicated model); the input
    batch is seeded by layer and rank (every rank works on its own images)."""
    W = synth.weights_kaiming(synth.rng(4, idx), L.M, L.Cin, L.k, L.k)
    x = synth.act_halfnormal(synth.rng(4, 5000 + idx + 100 * rank), (batch, L.H, L.H, L.Cin))
    return W, x


def layer_ops(L, batch):
    return 2 * L.macs(batch)


def layer_alg_bytes(L, batch, nP, nF4, n8):
    """Algorithmic bytes of one convolution launch: packed codes + 8 B/row metadata + each
    activation code the layer needs once (a strided 1x1 needs only the sampled pixels) + fp32 out."""
    K = L.K
    w = (nP + nF4) * K // 2 + n8 * K + 8 * L.M
    pix_in = L.Ho * L.Ho if (L.k == 1 and L.stride > 1) else L.H * L.H
    a = batch * pix_in * L.Cin
    o = 4 * batch * L.Ho * L.Ho * L.M
    return w + a + o


# ---------------------------------------------------------------------------- multi-GPU plumbing

def max_over_ranks(ms_local: float, world: int, device: str) -> float:
    """Slowest rank's time: the job is done when the last rank is (max over ranks, on `device`)."""
    if world <= 1:
        return float(ms_local)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_local], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tops(ops_per_gpu_step: int, world: int, ms_step: float) -> float:
    """Weak scaling over the batch: every rank runs the full stack on its own images, no exchange."""
    return world * ops_per_gpu_step / (ms_step * 1e-3) / 1e12


def launch_ranks(argv, gpus: int) -> int:
    """`bench.py --gpus N` started by hand (no WORLD_SIZE in the environment): start N ranks of this
    same command, one per GPU, under torch.distributed.run on the loop-back address, and return
    their exit code.  Rank 0 prints the one JSON line."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--standalone", "--local-addr", "127.0.0.1",
           "--nnodes=1", "--nproc-per-node", str(gpus), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def rank_env():
    """(world, rank, local_rank) from the launcher's environment; (1, 0, 0) when there is none."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


# ---------------------------------------------------------------------------- clocks

class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.idx = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def _size(self):
        try:
            return os.path.getsize(self.path)
        except Exception:
            return 0

    def mark(self):
        """Start of the timed regions: samples written before this point belong to the warm-up."""
        self.begin = self._size()

    def stop(self):
        if self.proc is None:
            return None
        try:
            time.sleep(0.05)                   # one more sampling period, so the last timed sample is on disk
            self.proc.terminate()
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, smax, reasons = [], [], set()
        try:
            data = open(self.path).read()
            begin = getattr(self, "begin", 0)
            # a sample that was being written when the region began or ended still counts
            begin = data.rfind("\n", 0, begin) + 1
            for line in data[begin:].splitlines():
                f = [t.strip() for t in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); smax.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if not sm:
            return None
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "reasons": sorted(reasons),
                "samples": len(sm), "period_ms": 20,
                "covers": "the device-resident timed region and the end-to-end timed region that follows it"}


# ---------------------------------------------------------------------------- our arm

def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2111_00153_b200 import binding as R

    world, rank, local = rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    R.lib()

    layers = layer_list()
    batch = args.batch
    stream = torch.cuda.current_stream()

    # ---- host inputs (seeded, synthetic) and device buffers
    H = []
    for i, L in enumerate(layers):
        W, x = host_layer(i, L, batch, rank)
        scheme, bits = R.rmsmp_assign_rows(W, RATIO)        # offline decision, not timed
        alpha = synth.alpha_rows(W)
        lay = R.rmsmp_layer_init(L.M, L.Cin, L.k, L.k, scheme, bits)
        H.append(dict(L=L, W=W, x=x, scheme=scheme, bits=bits, alpha=alpha, lay=lay))
    D = []
    for h in H:
        L = h["L"]
        N = batch * L.Ho * L.Ho
        D.append(dict(
            W=torch.from_numpy(h["W"]).cuda(), x=torch.from_numpy(h["x"]).cuda(),
            packed=torch.empty(h["lay"].packed_bytes, dtype=torch.uint8, device="cuda"),
            ws=torch.empty(R.rmsmp_workspace_bytes(h["lay"]), dtype=torch.int8, device="cuda"),
            codes=torch.empty(h["x"].shape, dtype=torch.int8, device="cuda"),
            y=torch.empty((N, L.M), dtype=torch.float32, device="cuda"), N=N))

    use_ws = (args.variant == "workspace")

    def conv(h, d, st):
        L = h["L"]
        if use_ws:
            R.rmsmp_conv_implicit_workspace(h["lay"], d["packed"], d["ws"], d["codes"], batch, L.H, L.H, L.stride,
                                            L.pad, st, d["y"], R.OUT_NM, None, stream=stream)
        else:
            R.rmsmp_conv_implicit_variant(h["lay"], d["packed"], d["codes"], batch, L.H, L.H, L.stride, L.pad, st,
                                          d["y"], R.OUT_NM, None, R.VARIANT_TENSOR, stream=stream)

    # Two streams: the weight path of a layer (quantize_pack + expand_weights: three small,
    # latency-bound launches) does not depend on its activations, so it runs on a side stream and
    # overlaps the activation quantizer / the previous layer's tail.  The convolution waits for
    # both; the next step's pack of a layer waits for this step's convolution of it (same buffers).
    side = torch.cuda.Stream() if args.streams >= 2 else None
    # --streams 3 (not the default: the convolution's own duration is then no longer measured in isolation):
    # the activation quantizer of layer i+1 also leaves the main stream and runs beside the convolution of layer i
    qs = torch.cuda.Stream() if args.streams == 3 else None
    qdone = [torch.cuda.Event() for _ in layers]
    ready = [torch.cuda.Event() for _ in layers]
    done = [torch.cuda.Event() for _ in layers]
    first_use = [True]

    def step(ev=None):
        for i, (h, d) in enumerate(zip(H, D)):
            ws_stream = side if side is not None else stream
            if side is not None:
                if first_use[0]:
                    side.wait_stream(stream)
                else:
                    side.wait_event(done[i])
            R.rmsmp_quantize_pack(d["W"], R.W_CONV_OIHW, h["lay"], h["scheme"], h["bits"], h["alpha"],
                                  R.POT_NEAREST, d["packed"], stream=ws_stream)
            if use_ws:
                R.rmsmp_expand_weights(h["lay"], d["packed"], d["ws"], stream=ws_stream)
            if side is not None:
                ready[i].record(side)
            if qs is not None:
                if first_use[0]:
                    qs.wait_stream(stream)
                else:
                    qs.wait_event(done[i])                   # the previous step's convolution has read these codes
                st = R.rmsmp_quantize_act(d["x"], d["x"].numel(), synth.ALPHA_ACT, R.ACT_U4, d["codes"], stream=qs)
                qdone[i].record(qs)
                stream.wait_event(qdone[i])
            else:
                st = R.rmsmp_quantize_act(d["x"], d["x"].numel(), synth.ALPHA_ACT, R.ACT_U4, d["codes"], stream=stream)
            if side is not None:
                stream.wait_event(ready[i])
            if ev is not None:
                ev[i][0].record(stream)
            conv(h, d, st)
            if ev is not None:
                ev[i][1].record(stream)
            if side is not None:
                done[i].record(stream)
        first_use[0] = False

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # the clock sampler starts before the warm-up (nvidia-smi needs a moment to deliver its first line);
    # its file position at the start of the timed region separates warm-up samples from timed ones
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    for d in D:
        assert R.rmsmp_last_device_status(d["packed"]) == R.OK

    # ---- device-resident timing
    evs = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in layers]
           for _ in range(args.steps)]
    barrier()
    if rank == 0:
        sampler.mark()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for k in range(args.steps):
        step(evs[k])
    t1.record(stream)
    barrier()
    ms_total = t0.elapsed_time(t1)
    ms_total = max_over_ranks(ms_total, world, "cuda")
    ms_step = ms_total / args.steps
    ops_step = sum(layer_ops(L, batch) for L in layers)
    conv_ms = np.array([[e[0].elapsed_time(e[1]) for e in evk] for evk in evs])   # [steps][layers]
    conv_ms_layer = conv_ms.mean(axis=0)
    alg = np.array([layer_alg_bytes(h["L"], batch, h["lay"].nP, h["lay"].nF4, h["lay"].n8) for h in H], dtype=np.float64)
    conv_total_ms = float(conv_ms_layer.sum())
    achieved_gbs = float(alg.sum() / (conv_total_ms * 1e-3) / 1e9)

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    if args.no_e2e:
        e2e_steps = 0
    pin = []
    for h, d in zip(H, D) if e2e_steps else ():
        pin.append(dict(W=torch.from_numpy(h["W"]).pin_memory(), x=torch.from_numpy(h["x"]).pin_memory(),
                        y=torch.empty(d["y"].shape, dtype=torch.float32).pin_memory()))

    # Three streams: host->device copies of the next layers run ahead on their own stream, the
    # device->host read of a layer's output follows its convolution on a third one, so the two
    # directions of the host link and the kernels overlap.  Everything is inside the timed region.
    s_in, s_out = (torch.cuda.Stream(), torch.cuda.Stream()) if e2e_steps else (None, None)
    in_ready = [torch.cuda.Event() for _ in layers]
    c_done = [torch.cuda.Event() for _ in layers]
    out_done = [torch.cuda.Event() for _ in layers]
    e2e_first = [True]

    def step_e2e():
        for i, (h, d, p) in enumerate(zip(H, D, pin)):
            if not e2e_first[0]:
                s_in.wait_event(c_done[i])               # the previous step's kernels have read W and x
            with torch.cuda.stream(s_in):
                d["W"].copy_(p["W"], non_blocking=True)
                d["x"].copy_(p["x"], non_blocking=True)
            in_ready[i].record(s_in)
        for i, (h, d, p) in enumerate(zip(H, D, pin)):
            stream.wait_event(in_ready[i])
            R.rmsmp_quantize_pack(d["W"], R.W_CONV_OIHW, h["lay"], h["scheme"], h["bits"], h["alpha"],
                                  R.POT_NEAREST, d["packed"], stream=stream)
            if use_ws:
                R.rmsmp_expand_weights(h["lay"], d["packed"], d["ws"], stream=stream)
            st = R.rmsmp_quantize_act(d["x"], d["x"].numel(), synth.ALPHA_ACT, R.ACT_U4, d["codes"], stream=stream)
            if not e2e_first[0]:
                stream.wait_event(out_done[i])           # the previous step's read of y has left
            conv(h, d, st)
            c_done[i].record(stream)
            s_out.wait_event(c_done[i])
            with torch.cuda.stream(s_out):
                p["y"].copy_(d["y"], non_blocking=True)
            out_done[i].record(s_out)
        e2e_first[0] = False

    if e2e_steps:
        step_e2e()
    barrier()
    t0.record(stream)
    if e2e_steps:
        s_in.wait_event(t0)
        s_out.wait_event(t0)
    for _ in range(e2e_steps):
        step_e2e()
    if e2e_steps:
        stream.wait_stream(s_in)
        stream.wait_stream(s_out)
    t1.record(stream)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    e2e_ms = max_over_ranks(t0.elapsed_time(t1), world, "cuda")
    e2e_ms_step = e2e_ms / max(e2e_steps, 1)
    h2d = int(sum(p["W"].numel() * 4 + p["x"].numel() * 4 for p in pin))
    d2h = int(sum(p["y"].numel() * 4 for p in pin))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peak_src = load_peaks()
    # tensor-bound part of the stack (the long-K layers that run on the two-CTA kernel) against the INT8
    # tensor-core rate measured in this run by the library's MMA-only loop (operands resident in shared memory)
    status_word = torch.zeros(4, dtype=torch.int32, device="cuda")
    i8_peak, _ = R.rmsmp_measure_mma_peak(status_word, False, 256, 20000)
    tb = [(layer_ops(h["L"], batch), float(ms)) for h, ms in zip(H, conv_ms_layer)
          if h["L"].K >= 2048 and h["L"].M % 256 == 0]
    tensor_tops = (sum(o for o, _ in tb) / (sum(m for _, m in tb) * 1e-3) / 1e12) if tb else None
    out = {
        "metric": METRIC, "value": whole_job_tops(ops_step, world, ms_step), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8xint8->int32 (w4/w8 a4), fp32 scale",
        "data": "synthetic",
        "config": {"workload": WORKLOAD if LAYER_FILTER is None else "subset:" + ",".join(sorted(LAYER_FILTER)), "batch_per_gpu": batch, "layers": len(layers),
                   "ops_per_step_per_gpu": ops_step, "l2": "inputs larger than L2 (every layer reads 13-205 MB and writes 6-205 MB)",
                   "step": "per layer: quantize_pack%s + quantize_act + conv_implicit (tensor cores, %s)" % ((" + expand_weights", "weights expanded once into scratch") if use_ws else ("", "weights expanded in shared memory per tile")),
                   "streams": args.streams},
        "clocks": clocks,
        "e2e": ({"value": whole_job_tops(ops_step, world, e2e_ms_step), "unit": UNIT, "ms_per_step": e2e_ms_step,
                 "steps": e2e_steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h} if e2e_steps else None),
        "gpu_launches": args.steps * len(layers) * (5 if use_ws else 4),
        "roofline": {"bound": "hbm", "kernel": "tensor_kernel + pair_kernel (conv_implicit)", "achieved": achieved_gbs,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved_gbs / peaks["hbm_gbs"],
                     "peak_source": peak_src,
                     "traffic": measured_traffic() if (batch == BATCH and use_ws and not args.layers) else None,
                     "algorithmic_bytes_per_step": float(alg.sum()), "kernel_ms_per_step": conv_total_ms,
                     "kernel_tops": ops_step / (conv_total_ms * 1e-3) / 1e12},
        "roofline_tensor": ({"bound": "tensor", "kernel": "pair_kernel (layers with K >= 2048 and M a multiple of 256)",
                             "achieved": tensor_tops, "peak": i8_peak, "unit": "TOP/s", "frac": tensor_tops / i8_peak,
                             "peak_source": "tcgen05.mma kind::i8 M=128 N=256 loop measured in this run (rmsmp_measure_mma_peak); "
                                            "2 x measured bf16 GEMM = %.0f" % (2 * peaks["bf16_tflops"]),
                             "layers": len(tb)} if tb and i8_peak > 0 else None),
        "roofline_weights": (weights_leg(R, torch, peaks) if (world == 1 and not args.no_weights_leg) else None),
        "per_config": (configs_leg(R, torch, peaks, i8_peak) if (world == 1 and not args.no_weights_leg and i8_peak > 0) else None),
        "second_workloads": (second_workloads_leg(R, torch, peaks, i8_peak) if (world == 1 and not args.no_weights_leg and i8_peak > 0) else None),
        "roofline_per_layer": binding_roof_summary(H, conv_ms_layer, alg, batch, peaks["hbm_gbs"], i8_peak, peaks),
        "per_layer": [{"name": h["L"].name, "M": h["L"].M, "K": h["L"].K, "N": d["N"], "ms": float(ms),
                       "tops": layer_ops(h["L"], batch) / (ms * 1e-3) / 1e12, "gbs": float(a / (ms * 1e-3) / 1e9)}
                      for h, d, ms, a in zip(H, D, conv_ms_layer, alg)],
    }
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(args.cpu_sample_batch)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def bert_large_stack(R, torch, ratio=RATIO, layers=24):
    """Config 5 as one cold stream: the linears of `layers` BERT-large encoder layers (4 x 1024x1024, 4096x1024,
    1024x4096 each), seeded N(0, 0.02) weights, rows assigned by variance rank, packed on the device."""
    out = []
    for l in range(layers):
        for j, (M, K) in enumerate(((1024, 1024),) * 4 + ((4096, 1024), (1024, 4096))):
            W = synth.weights_normal(synth.rng(5, 100 * l + j), (M, K))
            scheme, bits = R.rmsmp_assign_rows(W, ratio)
            lay = R.rmsmp_layer_init(M, K, 1, 1, scheme, bits)
            pk = torch.empty(lay.packed_bytes, dtype=torch.uint8, device="cuda")
            R.rmsmp_quantize_pack(torch.from_numpy(W).cuda(), R.W_LINEAR, lay, scheme, bits, synth.alpha_rows(W), R.POT_NEAREST, pk)
            out.append((lay, pk))
    torch.cuda.synchronize()
    return out


def configs_leg(R, torch, peaks, i8_peak):
    """Throughput of the other workload configurations (1: one small linear layer; 2: the 256->256 3x3
    convolution at 14x14, batch 32; 3: the four BERT-base linears at 4096 tokens), each through the
    call the benchmark's stack uses (weights expanded once into scratch, tensor cores), replayed 20
    times between two events.  Algorithmic bytes and ops as for the stack; every shape is reported
    against both roofs and names the one that binds it."""
    rows = []

    def one(cfg, name, M, Cin, k, stride, pad, B, H, kind):
        conv = k > 1 or H > 1
        g = synth.rng(6, M + Cin + k + B)
        W = synth.weights_kaiming(g, M, Cin, k, k) if conv else synth.weights_normal(g, (M, Cin)).reshape(M, Cin, 1, 1)
        scheme, bits = R.rmsmp_assign_rows(W, RATIO)
        lay = R.rmsmp_layer_init(M, Cin, k, k, scheme, bits)
        pk = torch.empty(lay.packed_bytes, dtype=torch.uint8, device="cuda")
        R.rmsmp_quantize_pack(torch.from_numpy(W).cuda(), R.W_CONV_OIHW, lay, scheme, bits, synth.alpha_rows(W), R.POT_NEAREST, pk)
        ws = torch.empty(R.rmsmp_workspace_bytes(lay), dtype=torch.int8, device="cuda")
        R.rmsmp_expand_weights(lay, pk, ws)
        Ho = (H + 2 * pad - k) // stride + 1
        N = B * Ho * Ho
        lo, hi = (0, 16) if kind == R.ACT_U4 else (-7, 8)
        act = torch.randint(lo, hi, (B, H, H, Cin), dtype=torch.int8, device="cuda")
        y = torch.empty((N, M), dtype=torch.float32, device="cuda")
        fn = lambda: R.rmsmp_conv_implicit_workspace(lay, pk, ws, act, B, H, H, stride, pad, 0.1, y, R.OUT_NM, None)
        for _ in range(5):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(20):
                fn()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) / 20)
        ms = float(np.median(ts))
        ops = 2 * M * Cin * k * k * N
        alg = (lay.nP + lay.nF4) * lay.K // 2 + lay.n8 * lay.K + 8 * M + B * H * H * Cin + 4 * N * M
        t_h, t_t = alg / (peaks["hbm_gbs"] * 1e9) * 1e3, ops / (i8_peak * 1e12) * 1e3
        rows.append({"config": cfg, "shape": name, "M": M, "K": Cin * k * k, "N": N, "us": ms * 1e3, "tops": ops / (ms * 1e-3) / 1e12,
                     "gbs": alg / (ms * 1e-3) / 1e9, "bound": "tensor" if t_t > t_h else "hbm", "frac": max(t_h, t_t) / ms,
                     "weights": "L2-resident replay"})

    one(1, "linear 256x512, 64 tokens", 256, 512, 1, 1, 0, 64, 1, R.ACT_U4)
    L = synth.CONFIG2_CONV
    one(2, "conv 256->256 3x3 on 14x14, batch 32", L.M, L.Cin, 3, 1, 1, 32, 14, R.ACT_U4)
    for nm, M, K in synth.BERT_BASE_LINEARS:
        one(3, "bert-base %s %dx%d, 4096 tokens" % (nm, M, K), M, K, 1, 1, 0, 4096, 1, R.ACT_S4)
    return rows


def second_workloads_leg(R, torch, peaks, i8_peak):
    """Layer shapes of the paper's other models (Section 4.1: MobileNet-v2, ResNet-50) and ResNet-18's first
    layer: depthwise 3x3 (CUDA cores), pointwise / bottleneck 1x1 and the 7x7 stride-2 first convolution
    with its three input channels stored as 16 (tensor cores).  Batch 64; 20 replays between two events."""
    rows = []

    def timed(fn):
        for _ in range(5):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(20):
                fn()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) / 20)
        return float(np.median(ts))

    def pack(W):
        scheme, bits = R.rmsmp_assign_rows(W, RATIO)
        lay = R.rmsmp_layer_init(W.shape[0], W.shape[1], W.shape[2], W.shape[3], scheme, bits)
        pk = torch.empty(lay.packed_bytes, dtype=torch.uint8, device="cuda")
        R.rmsmp_quantize_pack(torch.from_numpy(W).cuda(), R.W_CONV_OIHW, lay, scheme, bits, synth.alpha_rows(W), R.POT_NEAREST, pk)
        return lay, pk

    def record(name, lay, ms, ops, alg):
        t_h, t_t = alg / (peaks["hbm_gbs"] * 1e9) * 1e3, ops / (i8_peak * 1e12) * 1e3
        rows.append({"shape": name, "us": ms * 1e3, "tops": ops / (ms * 1e-3) / 1e12, "gbs": alg / (ms * 1e-3) / 1e9,
                     "bound": "tensor" if t_t > t_h else "hbm", "frac": max(t_h, t_t) / ms})

    B = 64
    for (C, H, stride) in ((144, 56, 1), (192, 28, 2), (960, 7, 1)):
        W = synth.weights_kaiming(synth.rng(7, C + H), C, 1, 3, 3)
        lay, pk = pack(W)
        Ho = (H + 2 - 3) // stride + 1
        act = torch.randint(0, 16, (B, H, H, C), dtype=torch.int8, device="cuda")
        y = torch.empty((B, Ho, Ho, C), dtype=torch.float32, device="cuda")
        ms = timed(lambda: R.rmsmp_conv_depthwise(lay, pk, act, B, H, H, stride, 1, 0.1, y))
        N = B * Ho * Ho
        record("mobilenet-v2 depthwise 3x3 C=%d %dx%d s%d B=%d" % (C, H, H, stride, B), lay, ms, 2 * 9 * C * N,
               lay.packed_bytes + B * H * H * C + 4 * N * C)
    for (name, M, Cin, k, stride, pad, H) in (("mobilenet-v2 pointwise 1x1 32->192 28x28", 192, 32, 1, 1, 0, 28),
                                              ("resnet-50 bottleneck 1x1 256->64 56x56", 64, 256, 1, 1, 0, 56),
                                              ("resnet-50 bottleneck 1x1 64->256 56x56", 256, 64, 1, 1, 0, 56),
                                              ("resnet-18 conv1 7x7 s2 (3 channels stored as 16) 224x224", 64, 16, 7, 2, 3, 224)):
        W = synth.weights_kaiming(synth.rng(7, M + Cin + k), M, Cin, k, k)
        if k == 7:
            W[:, 3:] = 0.0
        lay, pk = pack(W)
        ws = torch.empty(R.rmsmp_workspace_bytes(lay), dtype=torch.int8, device="cuda")
        R.rmsmp_expand_weights(lay, pk, ws)
        Ho = (H + 2 * pad - k) // stride + 1
        N = B * Ho * Ho
        act = torch.randint(0, 16, (B, H, H, Cin), dtype=torch.int8, device="cuda")
        y = torch.empty((N, M), dtype=torch.float32, device="cuda")
        ms = timed(lambda: R.rmsmp_conv_implicit_workspace(lay, pk, ws, act, B, H, H, stride, pad, 0.1, y, R.OUT_NM, None))
        real_cin = 3 if k == 7 else Cin
        record(name + " B=%d" % B, lay, ms, 2 * M * real_cin * k * k * N,
               (lay.nP + lay.nF4) * real_cin * k * k // 2 + lay.n8 * real_cin * k * k + 8 * M + B * H * H * real_cin + 4 * N * M)
    # the same first layer with its three channels as they are: patch matrix (rmsmp_im2col_codes), then the layer as
    # a linear layer over the patches (K = 147 padded to 160); the step is both kernels
    M, Cin, k, stride, pad, H = 64, 3, 7, 2, 3, 224
    W = synth.weights_kaiming(synth.rng(7, M + 16 + k), M, 16, k, k)[:, :3]
    K, ld = k * k * Cin, (k * k * Cin + 15) // 16 * 16
    Wl = np.zeros((M, ld, 1, 1), np.float32)
    Wl[:, :K, 0, 0] = W.transpose(0, 2, 3, 1).reshape(M, K)
    lay, pk = pack(Wl)
    ws = torch.empty(R.rmsmp_workspace_bytes(lay), dtype=torch.int8, device="cuda")
    R.rmsmp_expand_weights(lay, pk, ws)
    Ho = (H + 2 * pad - k) // stride + 1
    N = B * Ho * Ho
    act = torch.randint(0, 16, (B, H, H, Cin), dtype=torch.int8, device="cuda")
    cols = torch.empty((N, ld), dtype=torch.int8, device="cuda")
    y = torch.empty((N, M), dtype=torch.float32, device="cuda")

    def first_layer():
        R.rmsmp_im2col_codes(act, B, H, H, Cin, Cin, k, k, stride, pad, cols, ld)
        R.rmsmp_gemm_workspace(lay, pk, ws, cols, N, ld, 0.1, y, M, R.OUT_NM, None)
    ms = timed(first_layer)
    record("resnet-18 conv1 7x7 s2 (3 channels, patch matrix + linear layer) 224x224 B=%d" % B, lay, ms, 2 * M * K * N,
           (lay.nP + lay.nF4) * K // 2 + lay.n8 * K + 8 * M + B * H * H * Cin + 4 * N * M)
    return rows


def weights_leg(R, torch, peaks, tokens=(1, 8, 128), reps=5, launches=20, warm=50):
    """The weight-bound regime (config 5): the whole BERT-large stack (144 linears, ~160 MB of packed codes,
    more than L2) through ONE grouped tensor-core launch per pass, at a few token counts.  The plan is
    prepared once; a pass is one launch; `launches` passes run back to back between two events."""
    stack = bert_large_stack(R, torch)
    rows = []
    # unsigned codes (Eq. 1) at every token count, read as they are by the PoT tiles; one more row with signed
    # codes, which go through the E4M3 copy
    for N, signed in [(n, False) for n in tokens] + [(8, True)]:
        keep, items, alg, wbytes, ops = [], [], 0, 0, 0
        g = synth.rng(5, 9000 + N + (500 if signed else 0))
        for lay, pk in stack:
            M, K = lay.M, lay.Cin
            codes = synth.act_codes_uniform(g, (N, K))
            if signed:
                codes = (codes.astype(np.int16) - 8).astype(np.int8)
            act = torch.from_numpy(codes).cuda()
            y = torch.empty((N, M), dtype=torch.float32, device="cuda")
            keep.append((act, y))
            items.append((lay, pk, act, N, K, 0.1, y, M, None, 0 if signed else 1))
            w = (lay.nP + lay.nF4) * K // 2 + lay.n8 * K + 8 * M
            wbytes += w
            alg += w + N * K + 4 * N * M
            ops += 2 * M * K * N
        arr = R.make_gemm_items(items)
        table = torch.empty(R.rmsmp_grouped_plan_bytes(arr), dtype=torch.uint8, device="cuda")
        plan = R.rmsmp_gemm_grouped_prepare(arr, R.OUT_NM, table)
        for _ in range(warm):
            R.rmsmp_gemm_grouped_launch(plan)
        torch.cuda.synchronize()
        best = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(launches):
                R.rmsmp_gemm_grouped_launch(plan)
            b.record()
            torch.cuda.synchronize()
            best.append(a.elapsed_time(b) / launches)
        ms = float(np.median(best))
        for lay, pk in stack[:3]:
            assert R.rmsmp_last_device_status(pk) == R.OK
        rows.append({"tokens": N, "codes": "signed (E4M3 copy per launch)" if signed else "unsigned (act_nonneg)", "us": ms * 1e3, "gbs": alg / (ms * 1e-3) / 1e9, "frac": alg / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                     "tops": ops / (ms * 1e-3) / 1e12, "algorithmic_bytes": float(alg), "packed_weight_bytes": float(wbytes)})
        del keep, items, arr, table, plan
    head = rows[min(1, len(rows) - 1)]                    # the N = 8 row speaks for the regime
    return {"bound": "hbm", "kernel": "stream_kernel (rmsmp_gemm_grouped_launch: 144 BERT-large linears in one launch, ratio %d:%d:%d)" % RATIO,
            "achieved": head["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": head["frac"], "traffic": None,
            "at_tokens": head["tokens"], "rows": rows,
            "timing": "%d launches back to back between two events, median of %d; the packed weights (160 MB) exceed L2" % (launches, reps)}


def binding_roof_summary(H, ms_layer, alg_bytes, batch, hbm_gbs, i8_peak, peaks):
    """Each convolution against its OWN binding roof: the roofline time of a layer is the larger of
    bytes / HBM bandwidth and ops / INT8 tensor rate; the summary is sum(roofline time) / sum(time)."""
    if not i8_peak or i8_peak <= 0:
        return None
    roof_ms, kinds = [], []
    for h, a in zip(H, alg_bytes):
        t_h = a / (hbm_gbs * 1e9) * 1e3
        t_t = layer_ops(h["L"], batch) / (i8_peak * 1e12) * 1e3
        roof_ms.append(max(t_h, t_t))
        kinds.append("tensor" if t_t > t_h else "hbm")
    tot = float(np.sum(ms_layer))
    den = {"measured kind::i8 MMA loop": i8_peak, "2 x measured bf16 burst": 2 * peaks["bf16_tflops"],
           "2 x measured bf16 sustained": 2 * peaks.get("bf16_tflops_sustained", 0.0), "datasheet dense int8": 4500.0}
    tb = [(layer_ops(h["L"], batch), float(m)) for h, m, k in zip(H, ms_layer, kinds) if k == "tensor"]
    t_tops = (sum(o for o, _ in tb) / (sum(m for _, m in tb) * 1e-3) / 1e12) if tb else None
    return {"frac": float(np.sum(roof_ms)) / tot, "roofline_ms": float(np.sum(roof_ms)), "kernel_ms": tot,
            "layers": [{"name": h["L"].name, "bound": k, "frac": float(r / m)} for h, k, r, m in zip(H, kinds, roof_ms, ms_layer)],
            "tensor_bound_tops": t_tops,
            "tensor_bound_frac_by_denominator": ({n: (t_tops / v if v else None) for n, v in den.items()} if t_tops else None)}


TRAFFIC_NOTE = os.path.join(ROOT, "profiles", "resnet18_stack_dram_traffic.txt")
KERNEL_SOURCES = ("tensor.cu", "tensor2.cu", "common.cuh", "decode.cuh", "actq.cuh", "ptx.cuh", "tmap.cuh")


def kernel_sources_digest():
    """sha256 over the sources of the convolution kernels: ties a counter capture to the code it measured."""
    import hashlib
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2111_00153_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def measured_traffic():
    """DRAM bytes (read + write) of the 19 convolution launches of one step at batch 256, as the
    profiler's counters gave them, from the note the capture left -- or None when there is no note
    or the kernels' sources have changed since (stale counters are not reported)."""
    try:
        kv = dict(line.split(":", 1) for line in open(TRAFFIC_NOTE) if ":" in line and not line.startswith("#"))
        if kv["kernel_sources_sha256"].strip() != kernel_sources_digest():
            return None
        return float(kv["dram_bytes_per_step"])
    except Exception:
        return None


def write_traffic_note(csv_path):
    """Turns the profiler's launch list (ncu --csv with gpu__time_duration.sum, dram__bytes_read.sum and
    dram__bytes_write.sum per launch, taken on `bench.py --steps 2 --warmup 3 --no-e2e --no-cpu-baseline
    --no-weights-leg`) into the note measured_traffic() reads: the DRAM bytes of the 19 convolution launches
    of one whole step, tied to the digest of the kernels' sources."""
    import collections
    import csv
    rows = [r for r in csv.reader(open(csv_path)) if len(r) > 10]
    hdr = rows[0]
    ik, im, iv, iid = hdr.index("Kernel Name"), hdr.index("Metric Name"), hdr.index("Metric Value"), hdr.index("ID")
    per = collections.OrderedDict()
    for r in rows[1:]:
        per.setdefault(r[iid], {"name": r[ik]})[r[im]] = float(r[iv].replace(",", ""))
    conv = [v for v in per.values() if "tensor_kernel" in v["name"] or "pair_kernel" in v["name"]]
    first_form = conv[0]["name"] if conv else ""
    n_layers = len(layer_list())
    # a step starts with the first layer's kernel form after a different one (the l1 layers open the stack)
    l1 = next(v["name"] for v in conv if "pair_kernel" not in v["name"] and ", 3, " in v["name"])
    start = next(i for i in range(1, len(conv) - n_layers) if conv[i]["name"] == l1 and conv[i - 1]["name"] != l1)
    step = conv[start:start + n_layers]
    total = sum(v["dram__bytes_read.sum"] + v["dram__bytes_write.sum"] for v in step)
    us = sum(v["gpu__time_duration.sum"] for v in step) / 1e3
    with open(TRAFFIC_NOTE, "w") as f:
        f.write("# DRAM traffic of the %d convolution launches of one step (ResNet-18 stack, batch 256), from the profiler's\n" % n_layers)
        f.write("# launch list: ncu --metrics gpu__time_duration.sum,dram__bytes_read.sum,dram__bytes_write.sum --clock-control none\n")
        f.write("#   -s 200 -c 200 --csv --log-file %s python bench.py --steps 2 --warmup 3 --no-e2e --no-cpu-baseline --no-weights-leg\n" % csv_path)
        f.write("# then: python bench.py --write-traffic-note %s\n" % csv_path)
        f.write("kernel_sources_sha256: %s\n" % kernel_sources_digest())
        f.write("dram_bytes_per_step: %.0f\n" % total)
        f.write("conv_launches: %d\n" % len(step))
        f.write("conv_time_under_profiler_us: %.1f\n" % us)
    print(open(TRAFFIC_NOTE).read())


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                    "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", 0.0))}, "of measured"
        except Exception:
            pass
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "of fallback"


# ---------------------------------------------------------------------------- CPU oracle legs

def oracle_pass(batch, layers=None):
    """One pass of the oracle over the layer stack at `batch` images; returns (seconds, ops)."""
    from oracle import rmsmp_oracle as O
    layers = layers or layer_list()
    prepared = []
    for i, L in enumerate(layers):
        W, x = host_layer(i, L, batch)
        scheme, bits = O.assign_rows(W, RATIO)
        prepared.append((L, W, x, scheme, bits, synth.alpha_rows(W)))
    t0 = time.perf_counter()
    for L, W, x, scheme, bits, alpha in prepared:
        codes, st = O.quantize_act(x, synth.ALPHA_ACT, O.ACT_U4)
        O.layer_conv(W, scheme, bits, alpha, codes, st, L.stride, L.pad)
    dt = time.perf_counter() - t0
    return dt, sum(layer_ops(L, batch) for L in layers)


def cpu_baseline(sample_batch):
    from oracle import rmsmp_oracle as O
    O.build()
    oracle_pass(1)                       # page in / warm
    dt, ops = oracle_pass(sample_batch)
    return {"value": ops / dt / 1e12, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
            "sample": "the same 19-layer stack at batch %d of %d (%.1f s)" % (sample_batch, BATCH, dt)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import rmsmp_oracle as O
    O.build()
    t1, _ = oracle_pass(1)
    t1, _ = oracle_pass(1)
    n = args.steps + args.warmup
    b = int(max(1, min(32, 150.0 / (n * max(t1, 1e-3)))))
    for _ in range(args.warmup):
        oracle_pass(b)
    tot, ops = 0.0, 0
    for _ in range(args.steps):
        dt, o = oracle_pass(b)
        tot += dt
        ops += o
    val = ops / tot / 1e12
    sample = "the same 19-layer stack at batch %d of %d per step" % (b, BATCH)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": tot / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8xint8->int32 (w4/w8 a4), fp32 scale", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_check_ranks(args):
    """Plumbing self-check without a GPU (`--check-ranks`, any N): every rank joins a gloo group,
    draws the first layer's weights and its own input batch, and the ranks compare checksums and
    take the slowest of their (made-up) times.  Rank 0 prints what it found as one JSON line."""
    import torch
    import torch.distributed as dist
    world, rank, _ = rank_env()
    if world > 1:
        dist.init_process_group("gloo")
    L = synth.resnet18_convs()[-1]
    W, x = host_layer(0, L, 2, rank)
    mine = torch.tensor([float(np.abs(W).sum()), float(x.sum())], dtype=torch.float64)
    every = [torch.zeros_like(mine) for _ in range(world)]
    if world > 1:
        dist.all_gather(every, mine)
    else:
        every = [mine]
    ms = max_over_ranks(10.0 + 5.0 * rank, world, "cpu")
    if rank == 0:
        w = [float(t[0]) for t in every]
        xs = [float(t[1]) for t in every]
        print(json.dumps({"check": "ranks", "n_ranks": world, "weights_replicated": len(set(w)) == 1,
                          "inputs_differ": len(set(xs)) == world, "max_ms": ms,
                          "whole_job_tops_at_1e12_ops": whole_job_tops(10 ** 12, world, ms)}))
    if world > 1:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------- variant comparison

def run_suite(args):
    """Side-by-side timing of the contraction variants on the five workload configurations.
    Prints one JSON line per (shape, variant) and a markdown table; not the headline number."""
    import torch
    from paper_2111_00153_b200 import binding as R
    torch.cuda.set_device(0)
    peaks, peak_src = load_peaks()
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    i8_peak, _ = R.rmsmp_measure_mma_peak(status, False, 256, 20000)
    bf_peak, _ = R.rmsmp_measure_mma_peak(status, True, 256, 20000)
    print(json.dumps({"suite": "peaks", "int8_mma_tops_measured": i8_peak, "bf16_mma_tops_measured": bf_peak,
                      "hbm_gbs": peaks["hbm_gbs"], "hbm_source": peak_src}))
    rows = []

    def timed(fn, iters):
        for _ in range(3):
            fn(0)
        torch.cuda.synchronize()
        best = []
        for _ in range(5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(iters):
                fn(i)
            b.record()
            torch.cuda.synchronize()
            best.append(a.elapsed_time(b) / iters)
        return float(np.median(best)) * 1e3      # microseconds

    def prep(M, Cin, k, ratio, seed, conv):
        g = synth.rng(6, seed)
        W = synth.weights_kaiming(g, M, Cin, k, k) if conv else synth.weights_normal(g, (M, Cin)).reshape(M, Cin, 1, 1)
        scheme, bits = R.rmsmp_assign_rows(W, ratio)
        lay = R.rmsmp_layer_init(M, Cin, k, k, scheme, bits)
        pk = torch.empty(lay.packed_bytes, dtype=torch.uint8, device="cuda")
        R.rmsmp_quantize_pack(torch.from_numpy(W).cuda(), R.W_CONV_OIHW, lay, scheme, bits, synth.alpha_rows(W),
                              R.POT_NEAREST, pk)
        ws = torch.empty(R.rmsmp_workspace_bytes(lay), dtype=torch.int8, device="cuda")
        R.rmsmp_expand_weights(lay, pk, ws)
        return lay, pk, ws

    VAR = (("tensor_smem", R.VARIANT_TENSOR), ("tensor_workspace", "ws"), ("workspace_requant", "rq"),
           ("simt_dp4a", R.VARIANT_SIMT), ("shift_add", R.VARIANT_SHIFTADD))

    def want(tag):
        return not args.suite_filter or args.suite_filter in tag

    def bench_shape(cfg, name, M, Cin, k, stride, pad, B, H, ratio=RATIO, pool=1, only=None, iters=20):
        if not want(cfg):
            return
        conv = k > 1 or H > 1
        inst = [prep(M, Cin, k, ratio, 17 * i + M, conv) for i in range(pool)]
        Ho = (H + 2 * pad - k) // stride + 1
        N = B * Ho * Ho
        act = torch.randint(0, 16, (B, H, H, Cin), dtype=torch.int8, device="cuda")
        y = torch.empty((N, M), dtype=torch.float32, device="cuda")
        yc = torch.empty((N, M), dtype=torch.int8, device="cuda")
        lay0 = inst[0][0]
        ops = 2 * M * Cin * k * k * N
        pix_in = Ho * Ho if (k == 1 and stride > 1) else H * H
        alg = (lay0.nP + lay0.nF4) * lay0.K // 2 + lay0.n8 * lay0.K + 8 * M + B * pix_in * Cin + 4 * N * M
        for vname, v in VAR:
            if only and vname not in only:
                continue
            def fn(i, v=v):
                lay, pk, ws = inst[i % pool]
                if v == "rq":
                    R.rmsmp_conv_implicit_workspace_requant(lay, pk, ws, act, B, H, H, stride, pad, 0.1, 50.0, R.ACT_U4, yc)
                elif v == "ws":
                    R.rmsmp_conv_implicit_workspace(lay, pk, ws, act, B, H, H, stride, pad, 0.1, y, R.OUT_NM, None)
                else:
                    R.rmsmp_conv_implicit_variant(lay, pk, act, B, H, H, stride, pad, 0.1, y, R.OUT_NM, None, v)
            try:
                us = timed(fn, iters if v in ("ws", "rq", R.VARIANT_TENSOR) or ops < 2e10 else 3)
            except R.RmsmpError as e:
                print(json.dumps({"suite": cfg, "shape": name, "variant": vname, "error": str(e)}))
                continue
            alg_v = alg - 3 * N * M if v == "rq" else alg          # one code byte per output instead of four
            rec = {"suite": cfg, "shape": name, "M": M, "K": Cin * k * k, "N": N, "ratio": list(ratio), "variant": vname,
                   "us": us, "tops": ops / us / 1e6, "gbs": alg_v / us / 1e3, "frac_int8_peak": ops / us / 1e6 / i8_peak,
                   "frac_hbm": alg_v / us / 1e3 / peaks["hbm_gbs"], "weights": "cold pool of %d" % pool if pool > 1 else "warm"}
            rows.append(rec)
            print(json.dumps(rec))

    bench_shape("config1", "linear 256x512 N=64", 256, 512, 1, 1, 0, 64, 1)
    L = synth.CONFIG2_CONV
    bench_shape("config2", "conv 256->256 3x3 14x14 B=32", L.M, L.Cin, 3, 1, 1, 32, 14)
    for nm, M, K in synth.BERT_BASE_LINEARS:
        bench_shape("config3", "bert-base %s %dx%d N=4096" % (nm, M, K), M, K, 1, 1, 0, 4096, 1)
    for L in synth.resnet18_convs():
        if L.name in ("l1.conv3x3", "l2.conv3x3", "l2.down1x1_s2", "l3.conv3x3", "l4.conv3x3"):
            bench_shape("config4", "resnet18 %s B=256" % L.name, L.M, L.Cin, L.k, L.stride, L.pad, 256, L.H)
    for nm, M, K in synth.BERT_LARGE_LINEARS:
        for N in synth.BERT_LARGE_TOKENS:
            bench_shape("config5", "bert-large %s %dx%d N=%d" % (nm, M, K, N), M, K, 1, 1, 0, N, 1, pool=24,
                        only=("simt_dp4a", "shift_add") if N < 32 else None, iters=48)
    for ratio in synth.RATIO_SWEEP:
        bench_shape("config5", "bert-large ffn1 4096x1024 N=8 ratio %d:%d:%d" % ratio, 4096, 1024, 1, 1, 0, 8, 1,
                    ratio=ratio, pool=24, only=("simt_dp4a", "shift_add"), iters=48)
    # config 5 as the natural cold stream: the whole BERT-large stack (24 x six linears, ~158 MB of
    # packed weights, larger than L2) in ONE grouped launch; the table upload is part of the call.
    if want("grouped"):
        leg = weights_leg(R, torch, peaks)
        for r in leg["rows"]:
            rec = {"suite": "config5", "shape": "bert-large stack, 144 linears, N=%d, %s codes, one grouped launch (plan prepared once)" % (r["tokens"], r["codes"].split(" ")[0]),
                   "N": r["tokens"], "ratio": list(RATIO), "variant": "grouped_tensor", "us": r["us"], "tops": r["tops"], "gbs": r["gbs"],
                   "frac_int8_peak": r["tops"] / i8_peak, "frac_hbm": r["frac"], "weights": "cold stream"}
            rows.append(rec)
            print(json.dumps(rec))
    for N in (1, 8):
        if not want("grouped"):
            break
        keep, items, wbytes, ops, alg = [], [], 0, 0, 0
        for l in range(24):
            for (M, K) in ((1024, 1024),) * 4 + ((4096, 1024), (1024, 4096)):
                lay, pk, _ = prep(M, K, 1, RATIO, 1000 + 7 * l + M // 1000 + K // 500, False)
                act = torch.randint(0, 16, (N, K), dtype=torch.int8, device="cuda")
                yy = torch.empty((N, M), dtype=torch.float32, device="cuda")
                keep.append((lay, pk, act, yy))
                items.append((lay, pk, act, N, K, 0.1, yy, M, None))
                ops += 2 * M * K * N
                alg += (lay.nP + lay.nF4) * K // 2 + lay.n8 * K + 8 * M + N * K + 4 * N * M
        arr = R.make_gemm_items(items)
        table = torch.empty(R.rmsmp_grouped_table_bytes(len(items)), dtype=torch.uint8, device="cuda")
        us = timed(lambda i: R.rmsmp_gemm_grouped(arr, R.OUT_NM, table), 8)
        rec = {"suite": "config5", "shape": "bert-large stack, 144 linears, N=%d, one grouped launch" % N, "N": N,
               "ratio": list(RATIO), "variant": "grouped_dp4a", "us": us, "tops": ops / us / 1e6, "gbs": alg / us / 1e3,
               "frac_int8_peak": ops / us / 1e6 / i8_peak, "frac_hbm": alg / us / 1e3 / peaks["hbm_gbs"], "weights": "cold stream"}
        rows.append(rec)
        print(json.dumps(rec))
        del keep, items, arr, table
    print("\n| config | shape | variant | us | TOPS | GB/s | of INT8 peak | of HBM |")
    print("|---|---|---|---|---|---|---|---|")
    for r in rows:
        print("| %s | %s | %s | %.1f | %.1f | %.0f | %.1f %% | %.1f %% |" % (
            r["suite"], r["shape"], r["variant"], r["us"], r["tops"], r["gbs"], 100 * r["frac_int8_peak"], 100 * r["frac_hbm"]))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=BATCH)
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-sample-batch", type=int, default=128)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-weights-leg", action="store_true",
                    help="skip the weight-bound leg (the grouped BERT-large launch reported as roofline_weights)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--variant", default="workspace", choices=["workspace", "smem"],
                    help="tensor-core path: expand the weight codes once into scratch memory (default) "
                         "or in shared memory per tile")
    ap.add_argument("--streams", type=int, default=2, choices=[1, 2, 3],
                    help="2: each layer's weight path (pack, expand) runs on a side stream and overlaps the "
                         "activation path; 1: everything on one stream; 3: the activation quantizer too on a stream "
                         "of its own, beside the previous layer's convolution (kernel timings then overlap)")
    ap.add_argument("--suite", action="store_true",
                    help="side-by-side timing of the kernel variants on all five configurations (not the headline)")
    ap.add_argument("--suite-filter", default=None,
                    help="with --suite: only the rows whose configuration tag contains this text "
                         "(config1 .. config5, or 'grouped' for the one-launch BERT-large stack)")
    ap.add_argument("--weights-leg-only", default=None, metavar="TOKENS",
                    help="run only the weight-bound leg at this token count and print it (short: for profiler captures)")
    ap.add_argument("--second-workloads-only", action="store_true",
                    help="run only the depthwise / pointwise / bottleneck / first-layer shapes and print their rows (short: for profiler captures)")
    ap.add_argument("--write-traffic-note", default=None, metavar="CSV",
                    help="no GPU work: turn a profiler launch list into the DRAM-traffic note roofline.traffic is read from")
    ap.add_argument("--check-ranks", action="store_true",
                    help="no GPU work: the ranks check their seeding and the max-over-ranks exchange over gloo")
    ap.add_argument("--layers", default=None,
                    help="comma-separated layer names: run one instance of each (profiling runs)")
    args = ap.parse_args()
    if args.layers:
        global LAYER_FILTER
        LAYER_FILTER = set(args.layers.split(","))
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.suite:
        sys.exit(launch_ranks(sys.argv[1:], args.gpus))
    if args.write_traffic_note:
        write_traffic_note(args.write_traffic_note)
    elif args.weights_leg_only:
        import torch
        from paper_2111_00153_b200 import binding as R
        torch.cuda.set_device(0)
        peaks, _ = load_peaks()
        print(json.dumps(weights_leg(R, torch, peaks, tokens=(int(args.weights_leg_only),), reps=2, launches=3, warm=3)))
    elif args.second_workloads_only:
        import torch
        from paper_2111_00153_b200 import binding as R
        torch.cuda.set_device(0)
        peaks, _ = load_peaks()
        i8, _ = R.rmsmp_measure_mma_peak(torch.zeros(4, dtype=torch.int32, device="cuda"), False, 256, 20000)
        print(json.dumps(second_workloads_leg(R, torch, peaks, i8)))
    elif args.check_ranks:
        run_check_ranks(args)
    elif args.suite:
        run_suite(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
