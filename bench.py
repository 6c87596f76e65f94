#!/usr/bin/env python
"""Benchmark of the SDGP hot path: N:M pruning of dL/dO followed by the sparse tensor-core
data gradient, on synthetic tensors shaped like a network's convolution layers.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet9|gemm_large|fc_small|resnet50|regnetx]
                  [--scheme magnitude|rescaled|random] [--nm 2:4] [--impl ours|reference]

One step = every layer of the workload once: prune kernel + sparse dgrad kernel per layer
(the whole step replayed as one CUDA graph). Prints ONE JSON line.

  value      dense-equivalent TFLOP/s of the data gradient (2*M*N*K of the implicit GEMM,
             M = output pixels, N = Cin, K = R*S*Cout), prune time included, inputs resident.
  e2e        same metric with the step's dL/dO copied from pinned host memory and dL/dD copied
             back inside the timed region.
  roofline   the dominant kernel (sparse dgrad) against twice the measured dense bf16 peak.
  cpu_baseline  the CPU oracle on a bounded sample of the same workload.

With --impl reference the CPU oracle is the timed arm (there is no other implementation of
the paper's method to run); with more than one rank every rank runs an independent replica of
the workload (the path shards by batch with nothing to exchange).
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

from paper_2202_00774_b200 import inputs  # noqa: E402

SCHEMES = {"random": 0, "magnitude": 1, "rescaled": 2}
METRIC = "dgrad_dense_equiv_tflops"
UNIT = "TFLOP/s"


def workload_layers(name):
    if name == "resnet9":
        return inputs.resnet9_layers(512)
    if name == "gemm_large":
        c = inputs.GEMM_LARGE
        return [inputs.ConvLayer("gemm_16384x4096x4096", 1, 1, c["rows"], c["N"], c["K"], 1, 1, 1, 0)]
    if name == "fc_small":
        c = inputs.FC_SMALL
        return [inputs.ConvLayer("fc_256x512x256", 1, 1, c["rows"], c["N"], c["K"], 1, 1, 1, 0)]
    raise SystemExit("unknown workload " + name)


def layer_flops(l):
    return 2.0 * l.B * l.H * l.W * l.Cin * l.R * l.S * l.Cout


def layer_inputs(l, workload, seed, dtype="bf16"):
    if workload in ("resnet9", "resnet50"):
        dO, W = inputs.conv_layer_tensors(l, seed)
    else:
        dO, W = inputs.fc_tensors(l.W, l.Cout, l.Cin, seed)
        dO, W = dO.reshape(l.dO_shape()), W.reshape(l.W_shape())
    if dtype == "fp16":   # the same draw, re-encoded
        dO, W = inputs.bf16_bits_as_f16_bits(dO), inputs.bf16_bits_as_f16_bits(W)
    return dO, W


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of the seven sparse dgrad launches of one
# resnet9 two-pass step, from the ncu capture summarised in profiles/traffic_dgrad_sparse_resnet9.md,
# and the hash of the kernel sources it was taken with (the figure is dropped once they change).
NCU_TRAFFIC = {"workload": "resnet9", "mode": "two_pass", "bytes_per_step": 213.0e6, "sources_sha": "9e2b4e39f6d4dd4c"}
KERNEL_SOURCES = ["dgrad.cu", "ptx.cuh"]   # all the code of the non-fused data-gradient kernels


def kernel_sources_sha():
    """Hash of the data-gradient kernels' code with comments and blank lines left out (a comment edit is not a
    changed kernel)."""
    import hashlib
    import re
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2202_00774_b200", "csrc", f)) as fh:
            for line in fh:
                code = re.sub(r"//.*$", "", line).rstrip()
                if code.strip():
                    h.update(code.encode() + b"\n")
    return h.hexdigest()[:16]


def measured_traffic(workload, mode):
    if workload != NCU_TRAFFIC["workload"] or mode != NCU_TRAFFIC["mode"]:
        return None
    return NCU_TRAFFIC["bytes_per_step"] if kernel_sources_sha() == NCU_TRAFFIC["sources_sha"] else None


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=float(p["hbm_gbs"]), bf16=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


# ------------------------------------------------------------- CPU oracle arm


class OracleArm:
    """The CPU oracle on a bounded sample: per layer, prune `p` rows of dL/dO and evaluate the
    fp64 data gradient at `p` output pixels (the pruned neighbourhood is prepared once, outside
    the timed region). p is scaled so that a step lasts about `seconds`."""

    def __init__(self, layers, workload, n, m, scheme, dtype="bf16", channel=False):
        import oracle
        oracle.build()
        self.oracle = oracle
        self.channel = channel   # per-channel reading: magnitude survivors, one factor per channel inside the contraction
        if channel:
            scheme = oracle.MAGNITUDE
        self.n, self.m, self.scheme = n, m, scheme
        self.dt = oracle.FP16 if dtype == "fp16" else oracle.BF16
        # a slice of the workload large enough for ~30 s of oracle time: up to 256 images / 16384 rows
        self.layers = [inputs.ConvLayer(l.name, min(l.B, 256), l.H, min(l.W, 16384) if l.B == 1 and l.H == 1 else l.W,
                                        l.Cin, l.Cout, l.R, l.S, l.stride, l.pad) for l in layers]
        self.tensors = [layer_inputs(l, workload, 0, dtype) for l in self.layers]
        self.pruned = [oracle.prune(dO.reshape(-1, l.Cout), n, m, scheme, 0, want=("dense",), dtype=self.dt)["dense"].reshape(dO.shape)
                       for l, (dO, _) in zip(self.layers, self.tensors)]
        self.cores = oracle.omp_threads()

    def step(self, pixels):
        flops = 0.0
        self.last_pixels = []
        for l, (dO, W), pruned in zip(self.layers, self.tensors, self.pruned):
            p = int(max(1, min(pixels, l.B * l.H * l.W, l.B * l.P * l.Q)))
            self.last_pixels.append(p)
            self.oracle.prune(dO.reshape(-1, l.Cout)[:p], self.n, self.m, self.scheme, 0, want=("dense",), dtype=self.dt)
            ks = self.oracle.channel_scales(dO.reshape(-1, l.Cout)[:p], self.n, self.m, dtype=self.dt) if self.channel else None
            self.oracle.dgrad_conv2d(pruned, W, l.H, l.W, l.stride, l.pad, pixel_index=np.arange(p, dtype=np.int64),
                                     dtype=self.dt, k_scale=ks)
            flops += 2.0 * p * l.Cin * l.R * l.S * l.Cout
        return flops

    def pixels_for(self, seconds):
        # grow the probe until it is long enough to be dominated by the arithmetic, then scale
        probe, dt = 8, 0.0
        while True:
            t0 = time.perf_counter()
            self.step(probe)
            dt = max(time.perf_counter() - t0, 1e-6)
            if dt >= min(2.0, seconds / 4) or probe >= (1 << 20):   # long enough that fixed costs no longer count
                break
            probe *= 4
        return int(max(1, probe * seconds / dt))


def cpu_baseline(layers, workload, n, m, scheme, dtype="bf16", channel=False, target_s=24.0):
    arm = OracleArm(layers, workload, n, m, scheme, dtype, channel)
    pixels = arm.pixels_for(target_s)
    t0 = time.perf_counter()
    flops = arm.step(pixels)
    dt = time.perf_counter() - t0
    return dict(value=flops / dt / 1e12, unit=UNIT, cores=arm.cores, kind="oracle",
                sample="per layer %s dO rows pruned and as many output pixels of fp64 dgrad, %.1f s"
                       % (arm.last_pixels, dt))


def run_reference(args, layers):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n, m = [int(v) for v in args.nm.split(":")]
    arm = OracleArm(layers, args.workload, n, m, SCHEMES[args.scheme], args.dtype, args.mode == "channel")
    budget = min(20.0, 150.0 / max(1, args.steps + args.warmup))  # whole run stays within a few minutes
    pixels = arm.pixels_for(budget)
    for _ in range(args.warmup):
        arm.step(pixels)
    t0 = time.perf_counter()
    flops = 0.0
    for _ in range(args.steps):
        flops += arm.step(pixels)
    dt = time.perf_counter() - t0
    value = flops / dt / 1e12
    sample = "each step: per layer %s dO rows pruned and as many output pixels of fp64 dgrad" % (arm.last_pixels,)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "nm": args.nm, "scheme": args.scheme, "elements": args.dtype, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": arm.cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# -------------------------------------------------------------------- GPU arm


class ClockSampler:
    """nvidia-smi polled every 50 ms from construction to stop(); only the samples that fall inside a marked
    window (begin() ... end(): the timed regions) are reported."""
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        self.windows = []
        self.t_begin = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(device_index), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def begin(self):
        self.t_begin = time.time()

    def end(self):
        if self.t_begin is not None:
            self.windows.append((self.t_begin, time.time()))
            self.t_begin = None

    def stop(self):
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                stamp = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                clock, clock_max = float(f[1]), float(f[2])
            except ValueError:
                continue
            if self.windows and not any(a <= stamp <= b for a, b in self.windows):
                continue
            sm.append(clock)
            smax.append(clock_max)
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(smax)), reasons=sorted(reasons),
                       samples=len(sm))
        return out


def max_over_ranks(value, dist, device):
    """Largest `value` over all ranks (every rank gets it); identity without a process group."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def run_ours(args, layers):
    import torch
    import paper_2202_00774_b200 as sdgp

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    n, m = [int(v) for v in args.nm.split(":")]
    scheme = SCHEMES[args.scheme]
    pk = peaks()

    def dev16(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()

    DT = sdgp.FP16 if args.dtype == "fp16" else sdgp.BF16
    # patterns with more than two survivors in some 4-chunk have no 2:4 form: pruned dense copy + dense kernel
    masked = n > 2 and n != m
    if masked and args.mode != "two_pass":
        raise SystemExit("--mode %s needs n <= 2" % args.mode)
    step_flag = sdgp.FLAG_MASKED if masked else {"fused": sdgp.FLAG_FUSED, "channel": sdgp.FLAG_CHANNEL,
                                                 "two_pass": sdgp.FLAG_TWO_PASS}[args.mode]
    host_tensors = [layer_inputs(l, args.workload, rank, args.dtype) for l in layers]
    dO = [dev16(t[0]) for t in host_tensors]
    Wt = [dev16(t[1]) for t in host_tensors]
    dD = [torch.empty(l.dD_shape(), dtype=torch.int16, device="cuda") for l in layers]
    ws = [torch.empty(max(16, sdgp.sdgp_workspace_size_conv2d(l.B, l.H, l.W, l.Cin, l.Cout, l.R, l.S, l.stride, l.pad,
                                                              step_flag)),
                      dtype=torch.uint8, device="cuda") for l in layers]
    total_flops = sum(layer_flops(l) for l in layers)
    order = list(range(len(layers)))[::-1]  # backward pass: last layer first

    def sparse_step():
        for i in order:
            l = layers[i]
            sdgp.sdgp_dgrad_conv2d_typed(dO[i], Wt[i], dD[i], l.stride, l.pad, n, m, scheme, 1234, DT, workspace=ws[i],
                                         flags=step_flag)

    def dense_step():
        for i in order:
            l = layers[i]
            sdgp.sdgp_dgrad_conv2d_typed(dO[i], Wt[i], dD[i], l.stride, l.pad, n, m, scheme, 0, DT, flags=sdgp.FLAG_DENSE)

    def capture(fn):
        stream = torch.cuda.Stream()
        stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(stream):
            fn()  # warm-up outside capture: first calls configure kernel attributes
        torch.cuda.current_stream().wait_stream(stream)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        return g

    sampler = ClockSampler(torch.cuda.current_device()) if rank == 0 else None

    def timed(replay, steps, warmup, sample_clocks=False):
        for _ in range(warmup):
            replay()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if sampler and sample_clocks:
            sampler.begin()
        e0.record()
        for _ in range(steps):
            replay()
        e1.record()
        torch.cuda.synchronize()
        if sampler and sample_clocks:
            sampler.end()
        ms = e0.elapsed_time(e1)
        if dist is not None:
            ms = max_over_ranks(ms, dist, "cuda")
            dist.barrier()
        torch.cuda.synchronize()
        return ms

    g_sparse = capture(sparse_step)
    g_dense = capture(dense_step)

    # Clocks are sampled over the timed regions of the step and of the kernel-only graphs below (the step
    # itself may last only a few milliseconds; those graphs are replayed for at least 0.3 s each).
    ms_sparse = timed(g_sparse.replay, args.steps, args.warmup, sample_clocks=True)
    dense_steps = max(20, args.steps // 4)   # a replay lasts about 0.3 ms
    ms_dense = timed(g_dense.replay, dense_steps, max(3, args.warmup // 2))

    ms_per_step = ms_sparse / args.steps
    value = world * total_flops / (ms_per_step * 1e-3) / 1e12
    dense_value = world * total_flops / (ms_dense / dense_steps * 1e-3) / 1e12

    # The same chain with the prune inside the data-gradient kernel (one launch per layer), beside the two-pass step
    # of a default run: same tensors, same graph treatment, same number of timed replays as the dense twin.
    fused_chain = None
    if (args.mode == "two_pass" and not masked and n <= 2 and args.workload == "resnet9"
            and not (args.dtype == "fp16" and args.scheme == "rescaled")):
        def fused_step():
            for i in order:
                l = layers[i]
                sdgp.sdgp_dgrad_conv2d_typed(dO[i], Wt[i], dD[i], l.stride, l.pad, n, m, scheme, 1234, DT, flags=sdgp.FLAG_FUSED)
        g_fused = capture(fused_step)
        ms_fused = timed(g_fused.replay, dense_steps, max(3, args.warmup // 2))
        fused_value = world * total_flops / (ms_fused / dense_steps * 1e-3) / 1e12
        fused_chain = {"value": fused_value, "unit": UNIT, "ms_per_step": ms_fused / dense_steps,
                       "speedup_vs_dense": fused_value / dense_value, "steps": dense_steps,
                       "what": "the step as %d fused prune + sparse dgrad launches (SDGP_FLAG_FUSED), one CUDA graph" % len(layers)}

    # ---- the chain with the ReLU below every convolution (Section 2.1, Fig. 2: dL/dO comes out of the layer above;
    # Section 3.1: the unpruned tensor is kept for the weight gradient). Sparse side: the producer forms dL/dO from
    # the gradient above the ReLU and the activation, writes it and its compressed pruned copy in one pass, then the
    # sparse contraction. Dense side: a plain ReLU backward (the same kernel with n = m, which writes dL/dO only),
    # then the dense twin. Both sides pay for the pass over the gradient; each is one CUDA graph of 14 launches. ----
    relu_chain = None
    if (args.mode == "two_pass" and not masked and n <= 2 and args.workload == "resnet9" and not args.no_other_configs
            and all(l.Cout % 128 == 0 for l in layers)):
        act = [torch.randn(t.shape, device="cuda").clamp_(min=0).to(torch.float16 if args.dtype == "fp16" else torch.bfloat16)
               .view(torch.int16) for t in dO]
        grad = [torch.empty_like(t) for t in dO]
        cv = [torch.empty(l.B * l.P * l.Q * l.Cout // 2, dtype=torch.int16, device="cuda") for l in layers]
        cm = [torch.empty(l.B * l.P * l.Q * l.Cout // 16, dtype=torch.int16, device="cuda") for l in layers]

        def relu_sparse_step():
            for i in order:
                l = layers[i]
                sdgp.sdgp_relu_backward_prune(dO[i].view(-1, l.Cout), act[i].view(-1, l.Cout), n, m, scheme, 1234, dtype=DT,
                                              grad=grad[i].view(-1, l.Cout), values=cv[i], meta=cm[i])
                sdgp.sdgp_spmm_conv2d_typed(cv[i].view(l.B, l.P, l.Q, l.Cout // 2), cm[i].view(l.B, l.P, l.Q, l.Cout // 16),
                                            Wt[i], dD[i], l.stride, l.pad, DT)

        def relu_dense_step():
            for i in order:
                l = layers[i]
                sdgp.sdgp_relu_backward_prune(dO[i].view(-1, l.Cout), act[i].view(-1, l.Cout), 4, 4, scheme, 0, dtype=DT,
                                              grad=grad[i].view(-1, l.Cout))   # n == m: nothing pruned
                sdgp.sdgp_dgrad_conv2d_typed(grad[i], Wt[i], dD[i], l.stride, l.pad, n, m, scheme, 0, DT, flags=sdgp.FLAG_DENSE)

        g_rs, g_rd = capture(relu_sparse_step), capture(relu_dense_step)
        ms_rs = timed(g_rs.replay, dense_steps, max(3, args.warmup // 2)) / dense_steps
        ms_rd = timed(g_rd.replay, dense_steps, max(3, args.warmup // 2)) / dense_steps
        relu_chain = {"sparse_ms_per_step": ms_rs, "dense_ms_per_step": ms_rd, "speedup_vs_dense": ms_rd / ms_rs,
                      "steps": dense_steps,
                      "what": "every layer as [ReLU backward + prune in one pass (unpruned dL/dO kept), sparse contraction] "
                              "against [plain ReLU backward, dense twin], one CUDA graph each"}
        # the producer below a ReLU that follows a residual addition (two gradients added in the same pass), on the largest
        # tensor of the set: 3 reads + the unpruned dL/dO + values + positions = 9.125 B per element
        big = max(order, key=lambda i: dO[i].numel())
        lb = layers[big]
        skip = (torch.randn(dO[big].shape, device="cuda") * 0.5).to(torch.float16 if args.dtype == "fp16" else torch.bfloat16).view(torch.int16)
        g_res = capture(lambda: sdgp.sdgp_residual_relu_backward_prune(
            dO[big].view(-1, lb.Cout), skip.view(-1, lb.Cout), act[big].view(-1, lb.Cout), n, m, scheme, 1234, dtype=DT,
            grad=grad[big].view(-1, lb.Cout), values=cv[big], meta=cm[big]))
        ms_res = timed(g_res.replay, 50, 3) / 50
        res_gbs = dO[big].numel() * 9.125 / (ms_res * 1e-3) / 1e9
        relu_chain["residual_producer"] = {"layer": lb.name, "us": 1e3 * ms_res, "gbs": res_gbs, "frac_of_hbm": res_gbs / pk["hbm"],
                                           "bytes_per_element": 9.125}
        # ... and below a ReLU that is followed by 2 x 2 max pooling (the pooled gradient is scattered to each window's
        # maximum in the same pass): activation + a quarter-size gradient read, the unpruned dL/dO + values + positions
        # written = 5.625 B per element
        pooled = dO[big].view(lb.B, lb.P, lb.Q, lb.Cout)[:, : lb.P // 2, : lb.Q // 2].contiguous()
        g_pool = capture(lambda: sdgp.sdgp_maxpool_relu_backward_prune(
            pooled, act[big].view(lb.B, lb.P, lb.Q, lb.Cout), n, m, scheme, 1234, dtype=DT,
            grad=grad[big].view(lb.B, lb.P, lb.Q, lb.Cout), values=cv[big], meta=cm[big]))
        ms_pool = timed(g_pool.replay, 50, 3) / 50
        pool_gbs = dO[big].numel() * 5.625 / (ms_pool * 1e-3) / 1e9
        relu_chain["pool_producer"] = {"layer": lb.name, "us": 1e3 * ms_pool, "gbs": pool_gbs, "frac_of_hbm": pool_gbs / pk["hbm"],
                                       "bytes_per_element": 5.625}
        # ---- the chain with the producer each layer of ResNet-9 has above it (the normalisation layers left out): the
        # convolutions 64->128@32, 128->256@16 and 256->512@8 are followed by ReLU and 2 x 2 max pooling, the first and the
        # last of them with a residual block behind the pooling (two gradients reach the pooling's output); the other four
        # convolutions sit below a plain ReLU. Sparse side and dense side run the same producers (dense: n = m). ----
        if len(layers) == 7:
            pooled_layers = {0: True, 3: False, 4: True}    # layer index -> a residual block follows the pooling
            gp = {i: dO[i].view(layers[i].B, layers[i].P, layers[i].Q, layers[i].Cout)[:, : layers[i].P // 2, : layers[i].Q // 2]
                  .contiguous() for i in pooled_layers}
            gs = {i: (gp[i].view(torch.float16 if args.dtype == "fp16" else torch.bfloat16).float() * 0.5)
                  .to(torch.float16 if args.dtype == "fp16" else torch.bfloat16).view(torch.int16).flip(0).contiguous()
                  for i, res in pooled_layers.items() if res}

            def glue_step(sparse):
                for i in order:
                    l = layers[i]
                    nn, mm = (n, m) if sparse else (4, 4)   # n == m: nothing pruned
                    outs = dict(values=cv[i], meta=cm[i]) if sparse else {}
                    if i in pooled_layers:
                        sdgp.sdgp_maxpool_relu_backward_prune(gp[i], act[i].view(l.B, l.P, l.Q, l.Cout), nn, mm, scheme, 1234, dtype=DT,
                                                              grad=grad[i].view(l.B, l.P, l.Q, l.Cout), skip=gs.get(i), **outs)
                    else:
                        sdgp.sdgp_relu_backward_prune(dO[i].view(-1, l.Cout), act[i].view(-1, l.Cout), nn, mm, scheme, 1234, dtype=DT,
                                                      grad=grad[i].view(-1, l.Cout), **outs)
                    if sparse:
                        sdgp.sdgp_spmm_conv2d_typed(cv[i].view(l.B, l.P, l.Q, l.Cout // 2), cm[i].view(l.B, l.P, l.Q, l.Cout // 16),
                                                    Wt[i], dD[i], l.stride, l.pad, DT)
                    else:
                        sdgp.sdgp_dgrad_conv2d_typed(grad[i], Wt[i], dD[i], l.stride, l.pad, n, m, scheme, 0, DT, flags=sdgp.FLAG_DENSE)
            g_gs, g_gd = capture(lambda: glue_step(True)), capture(lambda: glue_step(False))
            ms_gs = timed(g_gs.replay, dense_steps, max(3, args.warmup // 2)) / dense_steps
            ms_gd = timed(g_gd.replay, dense_steps, max(3, args.warmup // 2)) / dense_steps
            relu_chain["resnet9_producers"] = {
                "sparse_ms_per_step": ms_gs, "dense_ms_per_step": ms_gd, "speedup_vs_dense": ms_gd / ms_gs,
                "what": "as above, but layers 0, 3, 4 below ReLU + 2 x 2 max pooling (0 and 4 with a second pooled gradient), "
                        "the others below a plain ReLU"}
            del gp, gs, g_gs, g_gd
        del act, grad, cv, cm, g_rs, g_rd, skip, g_res, pooled, g_pool

    # ---- per-kernel timing: the same step captured with timing events between the kernels
    # (event-record graph nodes), replayed with the same data and cache state as the timed step ----
    vals = [torch.empty(l.B * l.P * l.Q * l.Cout // (1 if masked else 2), dtype=torch.int16, device="cuda") for l in layers]
    metas = [torch.empty(l.B * l.P * l.Q * l.Cout // 16, dtype=torch.int16, device="cuda") for l in layers]

    kernel_scheme = SCHEMES["magnitude"] if args.mode == "channel" else scheme   # channel mode prunes by magnitude

    fused = args.mode == "fused"   # one kernel per layer: no separate prune launch, no compressed tensor

    def prune_only(i):
        l = layers[i]
        scheme = kernel_scheme
        if fused:
            return
        if masked:
            sdgp.sdgp_prune_typed(dO[i].view(-1, l.Cout), n, m, scheme, 1234, DT, dense=vals[i])
        else:
            sdgp.sdgp_prune_typed(dO[i].view(-1, l.Cout), n, m, scheme, 1234, DT, values=vals[i], meta=metas[i])

    def contraction_only(i):
        l = layers[i]
        if fused:
            sdgp.sdgp_dgrad_conv2d_typed(dO[i], Wt[i], dD[i], l.stride, l.pad, n, m, scheme, 1234, DT, flags=sdgp.FLAG_FUSED)
        elif masked:
            sdgp.sdgp_dgrad_conv2d_typed(vals[i].view(l.dO_shape()), Wt[i], dD[i], l.stride, l.pad, n, m, scheme, 0, DT,
                                         flags=sdgp.FLAG_DENSE)
        else:
            sdgp.sdgp_spmm_conv2d_typed(vals[i].view(l.B, l.P, l.Q, l.Cout // 2), metas[i].view(l.B, l.P, l.Q, l.Cout // 16),
                                        Wt[i], dD[i], l.stride, l.pad, DT)
    ev_s = [torch.cuda.Event(enable_timing=True, external=True) for _ in range(2 * len(layers) + 1)]
    ev_d = [torch.cuda.Event(enable_timing=True, external=True) for _ in range(len(layers) + 1)]

    def sparse_step_events():
        k = 0
        for i in order:
            l = layers[i]
            ev_s[k].record()
            prune_only(i)
            ev_s[k + 1].record()
            contraction_only(i)
            k += 2
        ev_s[k].record()

    def dense_step_events():
        for k, i in enumerate(order):
            l = layers[i]
            ev_d[k].record()
            sdgp.sdgp_dgrad_conv2d_typed(dO[i], Wt[i], dD[i], l.stride, l.pad, n, m, scheme, 0, DT, flags=sdgp.FLAG_DENSE)
        ev_d[len(order)].record()

    per_steps = max(3, min(args.steps, 30))
    prune_ms = [0.0] * len(layers)
    dgrad_ms = [0.0] * len(layers)
    dense_ms = [0.0] * len(layers)
    g_ev = capture(sparse_step_events)
    for it in range(per_steps + 3):
        g_ev.replay()
        torch.cuda.synchronize()
        if it >= 3:
            for k, i in enumerate(order):
                prune_ms[i] += 0.0 if fused else ev_s[2 * k].elapsed_time(ev_s[2 * k + 1])
                dgrad_ms[i] += ev_s[2 * k + 1].elapsed_time(ev_s[2 * k + 2])
    g_evd = capture(dense_step_events)
    for it in range(per_steps + 3):
        g_evd.replay()
        torch.cuda.synchronize()
        if it >= 3:
            for k, i in enumerate(order):
                dense_ms[i] += ev_d[k].elapsed_time(ev_d[k + 1])
    # ---- the seven sparse dgrad launches alone, back to back in one graph (their inputs are the
    # compressed tensors the event step left behind): no event node sits between the kernels, so
    # the graph time is the sum of the launch durations, gaps between launches included ----
    def dgrad_only_step():
        for i in order:
            contraction_only(i)

    g_dg = capture(dgrad_only_step)
    long_reps = int(max(per_steps, min(20000, 300.0 / max(ms_sparse / args.steps, 1e-3))))   # >= 0.3 s of replays
    ms_dgrad_total = timed(g_dg.replay, long_reps, 3, sample_clocks=True)
    ms_dgrad_only = ms_dgrad_total / long_reps

    # ---- the prune launches alone, the same way (their inputs, the seven dL/dO tensors, exceed L2) ----
    def prune_only_step():
        for i in order:
            prune_only(i)

    ms_prune_only = None
    if not fused:
        g_pr = capture(prune_only_step)
        ms_prune_only = timed(g_pr.replay, long_reps, 3, sample_clocks=True) / long_reps
    clocks = sampler.stop() if sampler else None
    status = sdgp.sdgp_last_device_error()
    if status != 0:
        raise SystemExit("device error: " + sdgp.status_string(status))
    bytes_per_element = 4.0 if masked else 3.125   # read 2 B; write a dense copy, or values + positions
    prune_bytes = sum(l.B * l.P * l.Q * l.Cout * bytes_per_element for l in layers)
    prune_gbs_events = prune_bytes * per_steps / (sum(prune_ms) * 1e-3) / 1e9 if not fused else None
    prune_gbs = prune_bytes / (ms_prune_only * 1e-3) / 1e9 if ms_prune_only else None
    dgrad_tflops_events = total_flops * per_steps / (sum(dgrad_ms) * 1e-3) / 1e12
    dgrad_tflops = total_flops / (ms_dgrad_only * 1e-3) / 1e12
    # Which measured peak the kernel-only figure is held against: the burst figure when the timed region is
    # shorter than a second or the sampled SM clock sat at its maximum (a kernel timed alone), the sustained
    # one otherwise (a seconds-long loop under the power cap). Both fractions are printed, and the one
    # against the data-sheet figure (2.25 PFLOP/s dense bf16, twice that for 2:4).
    mult = 1.0 if masked else 2.0   # binary16 has the same tensor-core rate as bf16
    at_max = bool(clocks and clocks.get("sm_mhz") and clocks["sm_mhz"] >= 0.97 * clocks["sm_max_mhz"])
    use_burst = (ms_dgrad_total < 1000.0) or at_max
    sparse_peak = mult * (pk["bf16"] if use_burst else pk["bf16_sustained"])
    peak_rule = ("burst: timed region %.0f ms%s" % (ms_dgrad_total, ", SM clock at max" if at_max else "") if use_burst
                 else "sustained: timed region %.0f ms, SM clock below max" % ms_dgrad_total)
    per_layer = [{"layer": l.name, "prune_us": 1e3 * prune_ms[i] / per_steps, "dgrad_us": 1e3 * dgrad_ms[i] / per_steps,
                  "dense_us": 1e3 * dense_ms[i] / per_steps,
                  "dgrad_dense_equiv_tflops": layer_flops(l) / (dgrad_ms[i] / per_steps * 1e-3) / 1e12,
                  "speedup_vs_dense": dense_ms[i] / (prune_ms[i] + dgrad_ms[i]),
                  "prune_gbs": (l.B * l.P * l.Q * l.Cout * bytes_per_element / (prune_ms[i] / per_steps * 1e-3) / 1e9
                                if not fused else None)}
                 for i, l in enumerate(layers)]

    # ---- end to end: dL/dO from pinned host memory, dL/dD back to the host, every step ----
    h_in = [torch.from_numpy(np.ascontiguousarray(t[0]).view(np.int16)).pin_memory() for t in host_tensors]
    h_out = [torch.empty(l.dD_shape(), dtype=torch.int16).pin_memory() for l in layers]
    h2d = sum(t.numel() * 2 for t in h_in)
    d2h = sum(t.numel() * 2 for t in h_out)

    # Three streams: host-to-device copies, kernels, device-to-host copies. Layer i's kernels wait for its
    # own input copy only, its output copy for its kernels only, so the two copy directions and the
    # kernels overlap inside a step; the step ends when all three streams have drained.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in layers]
    ev_done = [torch.cuda.Event() for _ in layers]

    def e2e_step():
        main = torch.cuda.current_stream()
        s_in.wait_stream(main)   # the previous step's kernels no longer read dL/dO
        s_out.wait_stream(main)
        with torch.cuda.stream(s_in):
            for i in order:
                dO[i].copy_(h_in[i], non_blocking=True)
                ev_in[i].record()
        for i in order:
            l = layers[i]
            main.wait_event(ev_in[i])
            sdgp.sdgp_dgrad_conv2d_typed(dO[i], Wt[i], dD[i], l.stride, l.pad, n, m, scheme, 1234, DT, workspace=ws[i],
                                         flags=step_flag)
            ev_done[i].record()
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[i])
                h_out[i].copy_(dD[i], non_blocking=True)
        main.wait_stream(s_in)
        main.wait_stream(s_out)

    e2e_steps = max(3, min(args.steps, 20))
    ms_e2e = timed(e2e_step, e2e_steps, 3)
    e2e_value = world * total_flops / (ms_e2e / e2e_steps * 1e-3) / 1e12

    # ---- one figure each for the two single-layer configurations (2:4 magnitude, two-pass, bf16), so that
    # they are measured by the same run as the headline: the small fully connected layer in microseconds,
    # the large GEMM as dense-equivalent TFLOP/s beside its dense twin, and the prune kernel on the large
    # GEMM's 134 MB dL/dO (larger than L2) in GB/s ----
    other_configs = None
    if rank == 0 and world == 1 and args.workload == "resnet9" and not args.no_other_configs:
        del h_in, h_out
        other_configs = {}
        for name in ("fc_small", "gemm_large"):
            l = workload_layers(name)[0]
            hdO, hW = layer_inputs(l, name, 0)
            xdO, xW = dev16(hdO), dev16(hW)
            xdD = torch.empty(l.dD_shape(), dtype=torch.int16, device="cuda")
            xws = torch.empty(max(16, sdgp.sdgp_workspace_size_conv2d(l.B, l.H, l.W, l.Cin, l.Cout, 1, 1, 1, 0, sdgp.FLAG_TWO_PASS)),
                              dtype=torch.uint8, device="cuda")
            xv = torch.empty(l.W * l.Cout // 2, dtype=torch.int16, device="cuda")
            xm = torch.empty(l.W * l.Cout // 16, dtype=torch.int16, device="cuda")
            # The small layer lasts a few microseconds, less than a graph launch costs the host: its graphs hold 50 calls
            # back to back, so that the figure is the device's time per call and not the host's launch rate.
            reps, inner = (40, 50) if name == "fc_small" else (20, 1)

            def repeated(fn, inner=inner):
                def body():
                    for _ in range(inner):
                        fn()
                return body
            g2 = capture(repeated(lambda: sdgp.sdgp_dgrad_conv2d(xdO, xW, xdD, 1, 0, 2, 4, SCHEMES["magnitude"], seed=1234, workspace=xws)))
            gd = capture(repeated(lambda: sdgp.sdgp_dgrad_conv2d(xdO, xW, xdD, 1, 0, 2, 4, SCHEMES["magnitude"], flags=sdgp.FLAG_DENSE)))
            gp = capture(repeated(lambda: sdgp.sdgp_prune(xdO.view(-1, l.Cout), 2, 4, SCHEMES["magnitude"], 1234, values=xv, meta=xm)))
            t2 = timed(g2.replay, reps, 3) / (reps * inner)
            td = timed(gd.replay, reps, 3) / (reps * inner)
            tp = timed(gp.replay, reps, 3) / (reps * inner)
            tf = None
            if name == "fc_small":   # one launch instead of two: the prune inside the data-gradient kernel
                gf = capture(repeated(lambda: sdgp.sdgp_dgrad_conv2d(xdO, xW, xdD, 1, 0, 2, 4, SCHEMES["magnitude"], seed=1234,
                                                                     flags=sdgp.FLAG_FUSED)))
                tf = timed(gf.replay, reps, 3) / (reps * inner)
                del gf
            fl = layer_flops(l)
            other_configs[name] = {
                "shape": "dO [%d x %d] . W [%d x %d]" % (l.W, l.Cout, l.Cout, l.Cin), "nm": "2:4", "scheme": "magnitude",
                "two_pass_us": 1e3 * t2, "dense_us": 1e3 * td, "prune_us": 1e3 * tp,
                "fused_us": (1e3 * tf) if tf else None, "fused_speedup_vs_dense": (td / tf) if tf else None,
                "value": fl / (t2 * 1e-3) / 1e12, "dense_tflops": fl / (td * 1e-3) / 1e12, "speedup_vs_dense": td / t2,
                "prune_gbs": l.W * l.Cout * 3.125 / (tp * 1e-3) / 1e9,
                "prune_frac_of_hbm": l.W * l.Cout * 3.125 / (tp * 1e-3) / 1e9 / pk["hbm"],
                "timing": "CUDA events around %d graph replays%s" % (
                    reps, "" if name == "gemm_large" else " of %d calls each; the tensors fit in L2, so this is a latency "
                                                          "figure, not a roofline one" % inner)}
            del xdO, xW, xdD, xws, xv, xm, g2, gd, gp
        if sdgp.sdgp_last_device_error() != 0:
            raise SystemExit("device error in the single-layer configurations")

    if rank == 0:
        base = (cpu_baseline(layers, args.workload, n, m, scheme, args.dtype, args.mode == "channel")
                if world == 1 and not args.no_cpu_baseline else None)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": args.dtype, "data": "synthetic",
            "config": {"workload": args.workload, "layers": len(layers), "nm": args.nm, "scheme": args.scheme,
                       "mode": "masked (pruned dense copy + dense kernel)" if masked else args.mode, "flops": "2*M*N*K of the implicit GEMM per layer",
                       "l2": "inputs larger than L2 (step touches %.0f MB)" % ((prune_bytes + d2h) / 1e6),
                       "launch": "one CUDA graph per step", "replicas": world},
            "speedup_vs_dense": value / dense_value, "dense_tflops": dense_value, "fused_chain": fused_chain,
            "relu_chain": relu_chain,
            "prune_gbs": prune_gbs, "prune_frac_of_hbm": (prune_gbs / pk["hbm"]) if prune_gbs else None,
            "prune_frac_of_nominal_8tbs": (prune_gbs / 8000.0) if prune_gbs else None,
            "prune_gbs_between_event_nodes": prune_gbs_events,
            "roofline": {"bound": "tensor",
                         "kernel": ("dense dgrad on the pruned copy (dgrad_halo_kernel<0,..>, dgrad_kernel<0,..>)" if masked
                                    else "fused prune + sparse dgrad (dgrad_halo_kernel<1,..,1>, dgrad_kernel<1,..,1>)" if fused
                                    else "sparse dgrad (dgrad_halo_kernel<1,..>, dgrad_kernel<1,..>)"),
                         "achieved": dgrad_tflops, "peak": sparse_peak, "unit": "TFLOP/s",
                         "frac": dgrad_tflops / sparse_peak, "peak_rule": peak_rule,
                         "frac_of_burst": dgrad_tflops / (mult * pk["bf16"]),
                         "frac_of_sustained": dgrad_tflops / (mult * pk["bf16_sustained"]),
                         "frac_of_nominal": dgrad_tflops / (mult * 2250.0),
                         "traffic": (measured_traffic(args.workload, args.mode)
                                     if not masked and args.dtype == "bf16" and args.nm == "2:4" and args.scheme == "magnitude"
                                     else None),
                         "traffic_unit": "DRAM bytes of the sparse dgrad launches of one step (ncu)",
                         "achieved_between_event_nodes": dgrad_tflops_events,
                         "note": "dense-equivalent FLOPs of the sparse dgrad launches of one step / the time of a "
                                 "graph holding exactly those launches back to back (CUDA events around %d replays); "
                                 "achieved_between_event_nodes: the same launches timed inside the full step by "
                                 "event nodes, each of which adds a few microseconds; "
                                 "peak = %d x %s dense bf16 (%s)" % (long_reps, 1 if masked else 2, pk["source"], peak_rule)},
            "per_layer": per_layer,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": {"fused": 1, "channel": 4}.get(args.mode, 2) * len(layers) * args.steps,
            "clocks": clocks,
        }
        if base is not None:
            line["cpu_baseline"] = base
        if other_configs is not None:
            line["configs"] = other_configs
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_layer_table(args):
    """--workload resnet50: every distinct bottleneck convolution of ResNet-50 at batch 256, one layer
    at a time (the tensors of all 23 shapes together would not be a step any trainer runs back to
    back with resident inputs): per layer the prune kernel, the sparse contraction, the fused kernel
    (groups of four only) and the dense twin, each timed by CUDA events around single launches with
    a write of 256 MB between launches (L2 flush), median of --steps launches (at most 50). The
    printed value weighs every shape by the number of times the network holds it."""
    import torch
    import paper_2202_00774_b200 as sdgp

    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    n, m = [int(v) for v in args.nm.split(":")]
    scheme = SCHEMES[args.scheme]
    pk = peaks()
    reps = max(5, min(args.steps, 50))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def dev16(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()

    def median_us(fn):
        for _ in range(max(3, min(args.warmup, 5))):
            fn()
        ts = []
        for _ in range(reps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(1e3 * e0.elapsed_time(e1))
        return float(np.median(ts))

    sampler = ClockSampler(torch.cuda.current_device())
    rows, launches = [], 0
    tot = dict(two_pass=0.0, best=0.0, dense=0.0, flops=0.0, prune=0.0, prune_bytes=0.0, spmm=0.0, chain_sparse=0.0, chain_dense=0.0)
    for l, count in inputs.resnet50_layers(256):
        dO_h, W_h = inputs.conv_layer_tensors(l, seed=0)
        dO, Wt = dev16(dO_h), dev16(W_h)
        del dO_h, W_h
        dD = torch.empty(l.dD_shape(), dtype=torch.int16, device="cuda")
        Cp = (l.Cout + 127) // 128 * 128
        ws = torch.empty(max(16, sdgp.sdgp_workspace_size_conv2d(l.B, l.H, l.W, l.Cin, l.Cout, l.R, l.S, l.stride, l.pad)),
                         dtype=torch.uint8, device="cuda")
        pix = l.B * l.P * l.Q
        vals = torch.empty(pix * l.Cout // 2, dtype=torch.int16, device="cuda")
        metas = torch.empty(pix * l.Cout // 16, dtype=torch.int16, device="cuda")
        def note(what):
            print("[%s] %s" % (l.name, what), file=sys.stderr, flush=True)

        note("two-pass")
        t_two = median_us(lambda: sdgp.sdgp_dgrad_conv2d(dO, Wt, dD, l.stride, l.pad, n, m, scheme, seed=1234, workspace=ws))
        note("prune")
        t_prune = median_us(lambda: sdgp.sdgp_prune(dO.view(-1, l.Cout), n, m, scheme, 1234, values=vals, meta=metas))
        t_spmm = None
        if Cp == l.Cout:
            note("sparse contraction")
            t_spmm = median_us(lambda: sdgp.sdgp_spmm_conv2d(vals.view(l.B, l.P, l.Q, l.Cout // 2),
                                                             metas.view(l.B, l.P, l.Q, l.Cout // 16), Wt, dD, l.stride, l.pad))
        t_fused = None
        if m == 4:
            note("fused")
            t_fused = median_us(lambda: sdgp.sdgp_dgrad_conv2d(dO, Wt, dD, l.stride, l.pad, n, m, scheme, seed=1234,
                                                               flags=sdgp.FLAG_FUSED))
        note("dense")
        t_dense = median_us(lambda: sdgp.sdgp_dgrad_conv2d(dO, Wt, dD, l.stride, l.pad, n, m, scheme, flags=sdgp.FLAG_DENSE))
        # The backward chain through the ReLU above the layer: the producer forms dL/dO from the gradient above the
        # ReLU and its activation and prunes it in the same pass (it also writes the unpruned dL/dO the weight
        # gradient needs), against a plain ReLU backward followed by the dense twin. Both sides pay for the pass.
        t_relu_prune = t_relu = None
        if t_spmm is not None and n <= 2:
            act = torch.randn(dO.shape, device="cuda").clamp_(min=0).to(torch.bfloat16).view(torch.int16)
            grad = torch.empty_like(dO)
            note("relu backward + prune")
            t_relu_prune = median_us(lambda: sdgp.sdgp_relu_backward_prune(dO.view(-1, l.Cout), act.view(-1, l.Cout), n, m, scheme, 1234,
                                                                          grad=grad.view(-1, l.Cout), values=vals, meta=metas))
            note("relu backward")
            t_relu = median_us(lambda: sdgp.sdgp_relu_backward_prune(dO.view(-1, l.Cout), act.view(-1, l.Cout), 4, 4, scheme, 0,
                                                                    grad=grad.view(-1, l.Cout)))
            launches += 2 * (reps + 3)
            del act, grad
        launches += (reps + 3) * (2 + 1 + (1 if t_spmm else 0) + (1 if t_fused else 0) + 1)
        status = sdgp.sdgp_last_device_error()
        if status != 0:
            raise SystemExit("device error: " + sdgp.status_string(status))
        fl = 2.0 * l.dense_macs
        bytes_dense = 2.0 * (pix * l.Cout + l.Cout * l.R * l.S * l.Cin + l.B * l.H * l.W * l.Cin)
        best = min(t for t in (t_two, t_fused) if t is not None)
        t_tensor = fl / (2.0 * pk["bf16_sustained"] * 1e12) * 1e6
        t_hbm = bytes_dense / (pk["hbm"] * 1e9) * 1e6
        rows.append({"layer": l.name, "count": count, "gflop": fl / 1e9, "two_pass_us": t_two, "prune_us": t_prune,
                     "spmm_us": t_spmm, "fused_us": t_fused, "dense_us": t_dense,
                     "speedup_two_pass": t_dense / t_two, "speedup_best": t_dense / best,
                     "speedup_spmm_alone": (t_dense / t_spmm) if t_spmm else None,
                     "bound": "tensor" if t_tensor >= t_hbm else "hbm",
                     "ideal_us": max(t_tensor, t_hbm), "frac_of_ideal_best": max(t_tensor, t_hbm) / best,
                     "prune_gbs": pix * l.Cout * 3.125 / (t_prune * 1e-6) / 1e9,
                     "relu_prune_us": t_relu_prune, "relu_us": t_relu,
                     "chain_sparse_us": (t_relu_prune + t_spmm) if t_relu_prune else None,
                     "chain_dense_us": (t_relu + t_dense) if t_relu else None,
                     "chain_speedup": ((t_relu + t_dense) / (t_relu_prune + t_spmm)) if t_relu_prune else None})
        if t_relu_prune:
            tot["chain_sparse"] += count * (t_relu_prune + t_spmm)
            tot["chain_dense"] += count * (t_relu + t_dense)
        tot["two_pass"] += count * t_two
        tot["best"] += count * best
        tot["dense"] += count * t_dense
        tot["flops"] += count * fl
        tot["prune"] += count * t_prune
        tot["prune_bytes"] += count * pix * l.Cout * 3.125
        del dO, Wt, dD, ws, vals, metas
        torch.cuda.empty_cache()
    clocks = sampler.stop()
    value = tot["flops"] / (tot["two_pass"] * 1e-6) / 1e12
    print(json.dumps({
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": 1, "steps": reps, "warmup": max(3, min(args.warmup, 5)),
        "ms_per_step": tot["two_pass"] / 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "resnet50", "layers": len(rows), "convolutions": sum(r["count"] for r in rows), "batch": 256,
                   "nm": args.nm, "scheme": args.scheme, "mode": "two_pass (per layer also fused and dense)",
                   "l2": "256 MB written between timed launches", "launch": "one launch per event pair, median"},
        "speedup_vs_dense": tot["dense"] / tot["two_pass"], "speedup_best_mode_vs_dense": tot["dense"] / tot["best"],
        "relu_chain": {"what": "per layer [ReLU backward + prune in one pass, then the sparse contraction] against [plain ReLU "
                               "backward, then the dense twin], over the shapes whose channel count needs no padding",
                       "sparse_us": tot["chain_sparse"], "dense_us": tot["chain_dense"],
                       "speedup": (tot["chain_dense"] / tot["chain_sparse"]) if tot["chain_sparse"] else None},
        "dense_tflops": tot["flops"] / (tot["dense"] * 1e-6) / 1e12,
        "prune_gbs": tot["prune_bytes"] / (tot["prune"] * 1e-6) / 1e9,
        "prune_frac_of_hbm": tot["prune_bytes"] / (tot["prune"] * 1e-6) / 1e9 / pk["hbm"],
        "per_layer": rows, "gpu_launches": launches, "clocks": clocks}))


def run_grouped_table(args):
    """--workload regnetx: every distinct convolution of the RegNetX-400MF body at batch 256 through
    sdgp_dgrad_conv2d_grouped (grouped 3x3 convolutions, channel counts 32 and 160 that are not multiples of 64), one
    layer at a time: two-pass, the dense twin and - where both channel counts are multiples of 64 - the fused
    kernel, each timed as in the ResNet-50 table (CUDA events around single calls, 256 MB written between them,
    median). FLOPs are the true ones of the grouped layer (Cin / groups input channels per output channel)."""
    import torch
    import paper_2202_00774_b200 as sdgp

    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    n, m = [int(v) for v in args.nm.split(":")]
    scheme = SCHEMES[args.scheme]
    pk = peaks()
    reps = max(5, min(args.steps, 50))
    warm = max(3, min(args.warmup, 5))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def median_us(fn):
        for _ in range(warm):
            fn()
        ts = []
        for _ in range(reps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(1e3 * e0.elapsed_time(e1))
        return float(np.median(ts))

    sampler = ClockSampler(torch.cuda.current_device())
    rows, launches = [], 0
    tot = dict(two_pass=0.0, dense=0.0, flops=0.0)
    for l, count in inputs.regnetx_400mf_layer_counts(256):
        dO_h, W_h = inputs.conv_layer_tensors(l, seed=0)
        dO = torch.from_numpy(np.ascontiguousarray(dO_h).view(np.int16)).cuda()
        Wt = torch.from_numpy(np.ascontiguousarray(W_h).view(np.int16)).cuda()
        del dO_h, W_h
        dD = torch.empty(l.dD_shape(), dtype=torch.int16, device="cuda")
        ws = torch.empty(sdgp.sdgp_workspace_size_conv2d_grouped(l.B, l.H, l.W, l.Cin, l.Cout, l.R, l.S, l.stride, l.pad, l.groups),
                         dtype=torch.uint8, device="cuda")

        def call(flags):
            sdgp.sdgp_dgrad_conv2d_grouped(dO, Wt, dD, l.stride, l.pad, l.groups, n, m, scheme, seed=1234, workspace=ws, flags=flags)

        print("[%s]" % l.name, file=sys.stderr, flush=True)
        t_two = median_us(lambda: call(sdgp.FLAG_TWO_PASS))
        t_dense = median_us(lambda: call(sdgp.FLAG_DENSE))
        t_fused = None
        if l.Cin % 64 == 0 and l.Cout % 64 == 0 and n <= 2:
            t_fused = median_us(lambda: call(sdgp.FLAG_FUSED))
        launches += (reps + warm) * (3 + 2 + (2 if t_fused else 0))   # filter expansion + (prune) + contraction
        status = sdgp.sdgp_last_device_error()
        if status != 0:
            raise SystemExit("device error: " + sdgp.status_string(status))
        fl = 2.0 * l.dense_macs
        pix = l.B * l.P * l.Q
        bytes_dense = 2.0 * (pix * l.Cout + l.Cout * l.R * l.S * (l.Cin // l.groups) + l.B * l.H * l.W * l.Cin)
        t_tensor = fl / (2.0 * pk["bf16_sustained"] * 1e12) * 1e6
        t_hbm = bytes_dense / (pk["hbm"] * 1e9) * 1e6
        rows.append({"layer": l.name, "count": count, "groups": l.groups, "gflop": fl / 1e9, "two_pass_us": t_two,
                     "fused_us": t_fused, "dense_us": t_dense, "speedup_two_pass": t_dense / t_two,
                     "bound": "tensor" if t_tensor >= t_hbm else "hbm", "ideal_dense_us": max(t_tensor, t_hbm),
                     "dense_frac_of_ideal": max(t_tensor, t_hbm) / t_dense})
        tot["two_pass"] += count * t_two
        tot["dense"] += count * t_dense
        tot["flops"] += count * fl
        del dO, Wt, dD, ws
        torch.cuda.empty_cache()
    clocks = sampler.stop()
    print(json.dumps({
        "metric": METRIC, "value": tot["flops"] / (tot["two_pass"] * 1e-6) / 1e12, "unit": UNIT, "n_gpus": 1, "steps": reps,
        "warmup": warm, "ms_per_step": tot["two_pass"] / 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "regnetx", "layers": len(rows), "convolutions": sum(r["count"] for r in rows), "batch": 256,
                   "nm": args.nm, "scheme": args.scheme, "mode": "two_pass (per layer also dense and, where it applies, fused)",
                   "flops": "true FLOPs of the grouped layers", "l2": "256 MB written between timed calls",
                   "launch": "one call per event pair (filter expansion included), median"},
        "speedup_vs_dense": tot["dense"] / tot["two_pass"],
        "dense_tflops": tot["flops"] / (tot["dense"] * 1e-6) / 1e12,
        "per_layer": rows, "gpu_launches": launches, "clocks": clocks}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet9", choices=["resnet9", "gemm_large", "fc_small", "resnet50", "regnetx"])
    ap.add_argument("--scheme", default="magnitude", choices=sorted(SCHEMES))
    ap.add_argument("--nm", default="2:4")
    ap.add_argument("--mode", default="two_pass", choices=["two_pass", "fused", "channel"],
                    help="two_pass: prune kernel + sparse dgrad kernel per layer; fused: one kernel prunes and contracts; "
                         "channel: two-pass under the per-channel reading of the L1 rescale (implies --scheme rescaled)")
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp16"],
                    help="element type of dL/dO, W and dL/dD (fp32 accumulation either way)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the quick figures for the small fully connected layer and the large GEMM (key `configs`)")
    args = ap.parse_args()
    if args.mode == "channel":
        args.scheme = "rescaled"
    if args.workload in ("resnet50", "regnetx"):
        if args.impl == "reference" or args.gpus != 1:
            raise SystemExit("--workload %s is a single-GPU per-layer table of this implementation" % args.workload)
        return run_layer_table(args) if args.workload == "resnet50" else run_grouped_table(args)
    layers = workload_layers(args.workload)
    if args.impl == "reference":
        run_reference(args, layers)
    else:
        run_ours(args, layers)


if __name__ == "__main__":
    main()
