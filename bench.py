#!/usr/bin/env python
"""Benchmark of the DARK-attention hot path: forward + backward tokens/s at N = 8192 on B200.

One step = one forward and one backward call of the whole hot path (feature maps, chunked causal
scan, dQ/dK/dV/dM) over one batch of the synthetic workload. Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload headline]

With --gpus N > 1 and no launcher environment the script starts itself again under torch.distributed.run, one
rank per GPU; every rank processes its own batch (weak scaling) with the parameters M and W of rank 0's
workload, and the per-head gradient of M is all-reduced over NCCL, as in data-parallel training.
`--impl reference` times the float64 CPU oracle on the host cores (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "DARK-attention fwd+bwd tokens/s"
UNIT = "tokens/s"
MIN_TIMED_SECONDS = 2.0          # the K timed steps are repeated until this much device time has been measured


def ncu_traffic_per_token_head():
    """DRAM bytes (read + write) per (token, head) of the scan kernels from their ncu capture on the small profiling
    workload, kept next to the capture's summary; traffic is proportional to the (token, head) count. A kernel that
    changed since its capture has no entry."""
    path = os.path.join(ROOT, "profiles", "scan_kernels_d128_small.traffic.json")
    try:
        with open(path) as f:
            return json.load(f)
    except (OSError, ValueError):
        return {}


def flops_per_token_head(d, r, m, dv, C, causal, backward):
    """Algorithmic floating-point operations per (token, head); intra-chunk terms count the lower
    triangle only. Backward: with the forward pass's stash the state before each chunk and the key features are read
    back, so the backward pass forms the query features only (half of the feature maps' flops) and its state terms
    are dO S^T, R += A^T dO, V R^T and Bf R: 8 m dv. The non-causal backward forms both sides' features again."""
    feat = 2 * (2 * d * r + 2 * r * m)                 # both sides: x~ = M x and u = W x~
    fwd = feat + 4 * m * dv + ((C + 1) * (m + dv) if causal else 0)
    if not backward:
        return fwd
    refeat = feat // 2 if causal else feat
    bwd = refeat + 8 * m * dv + ((C + 1) * (3 * m + 2 * dv) if causal else 0) + 4 * m * r + 8 * r * d
    return fwd + bwd


def bytes_per_token_head(d, dv, backward, e=2):
    fwd = (2 * d + 2 * dv) * e                          # Q, K, V in; O out
    return fwd + ((4 * d + 4 * dv) * e if backward else 0)   # + Q,K,V,dO in; dQ,dK,dV out (+O)


def exps_per_token_head(m, causal, backward):
    return 2 * m + ((m if causal else 2 * m) if backward else 0)


def kernel_work(d, r, m, dv, C, nslab, causal):
    """Algorithmic work per (token, head) of each kernel of the tensor-core path: (flops, exps, bytes,
    bound). The scan kernels split the step's total of flops_per_token_head() between them: the causal
    query-side backward kernel is charged the query features' recompute (both backward kernels read the key features
    the forward scan stored, the key-side one also the query features the query-side one stored), each backward kernel
    half of the feature-map backward; bytes count what the kernel has to move once (inputs, outputs, and the stashed
    tiles it reads or writes). The helper kernels are HBM-bound and are charged the tensors they read and write once."""
    feat = 2 * (2 * d * r + 2 * r * m)
    tri = C + 1
    e = 2
    k = {
        "tc_fwd_causal_kernel": (feat + 4 * m * dv + tri * (m + dv), 2 * m, (2 * d + 2 * dv) * e, "tensor"),
        "tc_fwd_keys_kernel": (feat // 2 + 2 * m * dv, m, (d + dv) * e, "tensor"),
        "tc_fwd_queries_kernel": (feat // 2 + 2 * m * dv, m, (d + dv) * e, "tensor"),
        "tc_bwd_q_kernel": (feat // 2 + 2 * m * dv + tri * (m + dv) + 2 * m * r + 4 * r * d, m,
                            (2 * d + 2 * dv + 2 * m) * e + m * dv * e // C, "tensor"),
        "tc_bwd_k_kernel": (6 * m * dv + tri * (2 * m + dv) + 2 * m * r + 4 * r * d, 0, (2 * d + 3 * dv + 2 * m) * e, "tensor"),
        "tc_bwd_nc_q_kernel": (feat // 2 + 4 * m * dv + 2 * m * r + 4 * r * d, m, (2 * d + dv) * e, "tensor"),
        "tc_bwd_nc_k_kernel": (feat // 2 + 4 * m * dv + 2 * m * r + 4 * r * d, m, (2 * d + 2 * dv) * e, "tensor"),
        "tc_bwd_finish_k_kernel": (6 * r * d, 0, 3 * d * e, "hbm"),
        "tc_key_prepass_kernel": (2 * r * d + 2 * d * m, 0, d * e + 4, "hbm"),
        "combine_kernel": (0, 0, (nslab * dv + dv) * e + nslab * 32, "hbm"),
        "delta_kernel": (0, 0, 2 * dv * e + 4, "hbm"),
    }
    return k


def launcher_command(argv, gpus, port=None):
    """The command that starts this script once per GPU of one node."""
    port = port or (29500 + os.getpid() % 2000)
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid, self.rows, self.proc = uuid, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
                for n, v in zip(names, r[4:8]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return {"hbm_gbs": j["hbm_gbs"], "bf16_tflops": j["bf16_tflops"],
                "bf16_tflops_sustained": j.get("bf16_tflops_sustained", j["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def oracle_step(ref, sub, wl):
    ref.forward(sub.Q, sub.K, sub.V, sub.M, sub.W, causal=wl.causal)
    if wl.backward:
        ref.backward(sub.Q, sub.K, sub.V, sub.M, sub.W, sub.dO, causal=wl.causal)


def oracle_sample(wl, inputs, ref):
    cores = ref.num_threads()
    B, H = wl.B, wl.H
    P = max(1, min(cores, B * H, 64))
    pairs = [((i * 7) % B, (i * 5) % H) for i in range(B * H)]
    seen, use = set(), []
    for p in pairs:
        if p not in seen:
            seen.add(p); use.append(p)
        if len(use) == P:
            break
    sub = inputs.generate(wl, pairs=use)
    return sub, use, min(cores, len(use))


def run_reference(args, wl):
    """The oracle, as it stands, on the host cores: each step = forward+backward of a bounded sample."""
    from oracle import ref
    from paper_2603_04127_b200 import inputs
    if int(os.environ.get("RANK", "0")) != 0:
        return
    sub, use, cores = oracle_sample(wl, inputs, ref)
    for _ in range(args.warmup):
        oracle_step(ref, sub, wl)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(ref, sub, wl)
    dt = (time.perf_counter() - t0) / args.steps
    tokens = len(use) * wl.N / wl.H                    # (token, head) pairs processed / heads per token
    val = tokens / dt
    sample = f"{len(use)} of {wl.B * wl.H} (batch, head) pairs at full N={wl.N}, forward+backward, float64"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_config(wl):
    B, H, N, d, r, m, dv = wl.dims()
    return {"workload": f"{wl.name}: B={B} H={H} N={N} d={d} r={r} m={m} dv={dv} "
                        f"{'causal (chunk 128)' if wl.causal else 'non-causal'} "
                        f"{'forward+backward' if wl.backward else 'forward'} {wl.dtype}",
            "l2": "inputs larger than L2 (Q,K,V,dO total %.0f MB)" % ((3 * B * H * N * d + B * H * N * dv) * 2 / 1e6)}


def extra_configs(torch, binding, inputs, peaks, tensor_peak, exclude, steps=20):
    """Short device-timed runs of the other workloads (the five configurations and the non-causal headline shape), so
    that one bench line carries the whole table: ms per step, tokens/s, and the whole step's algorithmic flops against
    the tensor peak."""
    out = {}
    stream = torch.cuda.current_stream()
    for name in ("c1", "c2", "c3", "c4", "c5", "headline", "headline_nc"):
        if name == exclude:
            continue
        wl = inputs.WORKLOADS[name]
        B, H, N, d, r, m, dv = wl.dims()
        t = inputs.generate(wl)
        dt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
        dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()
        Q, K, V, M, W = (dev(x) for x in (t.Q, t.K, t.V, t.M, t.W))
        G = dev(t.dO) if wl.backward else None
        del t
        O = torch.empty_like(V)
        plan = binding.darkattn_plan(B, H, N, d, m, r=r, dv=dv, dtype=binding.BF16 if wl.dtype == "bf16" else binding.F32, causal=wl.causal)
        ws = plan.alloc_workspace()
        saved = torch.empty(plan.saved_bytes, dtype=torch.uint8, device="cuda") if (plan.saved_bytes and wl.backward) else None
        if wl.backward:
            dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
            dM = torch.empty(M.shape, dtype=torch.float32, device="cuda")

        def step():
            binding.darkattn_forward(plan, Q, K, V, M, W, O, ws, saved=saved, stream=stream)
            if wl.backward:
                binding.darkattn_backward(plan, Q, K, V, M, W, O, G, dQ, dK, dV, dM, ws, saved=saved, stream=stream)

        for _ in range(3):
            step()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(steps):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        ok = binding.darkattn_last_device_status(plan, ws) == binding.OK
        flops = flops_per_token_head(d, r, m, dv, 128, wl.causal, wl.backward) * B * H * N
        entry = {"workload": workload_config(wl)["workload"], "path": {1: "simt", 2: "tensor"}[plan.path], "ms_per_step": ms,
                 "tokens_per_s": B * N / (ms * 1e-3), "steps": steps, "device_status_ok": ok,
                 "achieved_tflops": flops / (ms * 1e-3) / 1e12}
        if plan.path == binding.PATH_TENSOR:
            entry["frac_of_tensor_peak"] = entry["achieved_tflops"] / tensor_peak
        out[name] = entry
        plan.destroy()
        del Q, K, V, M, W, G, O, ws, saved
        if wl.backward:
            del dQ, dK, dV, dM
        torch.cuda.empty_cache()
    return out


def decode_benchmark(torch, binding, inputs, peaks, B=4, H=16, d=128, m=256, dv=128, steps=200):
    """The single-token decode step on B H = 64 (batch, head) pairs: bound by the traffic of the running state, which it
    reads and writes once (m dv 4 bytes each way per pair, plus z); reported as GB/s against the measured copy bandwidth."""
    g = torch.Generator(device="cuda").manual_seed(1)
    rn = lambda *s: torch.randn(*s, device="cuda", generator=g).to(torch.bfloat16)
    q, k, v = rn(B, H, d), rn(B, H, d), rn(B, H, dv)
    M = (torch.eye(d, device="cuda")[None] + 0.1 * torch.randn(H, d, d, device="cuda", generator=g) / d ** 0.5).to(torch.bfloat16)
    W = rn(m, d)
    S = torch.zeros(B, H, m, dv, dtype=torch.float32, device="cuda")
    z = torch.zeros(B, H, m, dtype=torch.float32, device="cuda")
    o = torch.empty(B, H, dv, dtype=torch.bfloat16, device="cuda")
    plan = binding.darkattn_plan(B, H, 128, d, m, dv=dv, dtype=binding.BF16, causal=True)
    stream = torch.cuda.current_stream()
    for _ in range(5):
        binding.darkattn_decode_step(plan, q, k, v, M, W, S, z, o, stream=stream)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(steps):
        binding.darkattn_decode_step(plan, q, k, v, M, W, S, z, o, stream=stream)
    e1.record(stream)
    torch.cuda.synchronize()
    us = 1e3 * e0.elapsed_time(e1) / steps
    nbytes = B * H * (2 * m * dv * 4 + 2 * m * 4) + (H * d * d + m * d) * 2
    plan.destroy()
    state_mb = B * H * m * dv * 4 / 1e6
    note = ("at this size the state, %.0f MB, stays in L2: launch- and latency-bound" % state_mb if state_mb < 100
            else "state of %.0f MB, larger than L2" % state_mb)
    return {"workload": f"decode step: B={B} H={H} d={d} m={m} dv={dv} bf16, state fp32", "us_per_step": us, "launches_per_step": 1,
            "bound": "hbm (state read and written once; " + note + ")",
            "achieved": nbytes / (us * 1e-6) / 1e9, "unit": "GB/s", "peak": peaks["hbm_gbs"],
            "frac": nbytes / (us * 1e-6) / 1e9 / peaks["hbm_gbs"], "tokens_per_s": B / (us * 1e-6)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="headline")
    ap.add_argument("--path", type=int, default=0, help="0 auto, 1 SIMT, 2 tensor")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernel-times", action="store_true")
    ap.add_argument("--no-extra-configs", action="store_true", help="skip the short runs of the other workloads and of the decode step")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_SECONDS, help="device time to measure at least (the K steps are repeated)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2603_04127_b200 import inputs
    workloads = dict(inputs.WORKLOADS)
    # for profiler captures: the headline's per-head shape on fewer, shorter sequences, one CTA per SM (2 * 37 heads * 2 slabs
    # = 148), inputs still larger than L2, small enough for a full counter capture
    workloads["profile_small"] = inputs.Workload("profile_small", 3, 2, 37, 2048, 128, 256, "bf16", True, backward=True, rho=0.95)
    wl = workloads[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
        return

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not started by a launcher: start one rank per GPU (NCCL's own log lines stay on)
        sys.exit(subprocess.call(launcher_command(sys.argv[1:], args.gpus)))

    import torch
    import torch.distributed as dist

    from paper_2603_04127_b200 import sharding
    rank, world, local = sharding.env_rank_world()
    if not torch.cuda.is_available():
        sys.exit(f"bench.py: rank {rank} of {world}: no CUDA device (the benchmark has no CPU path)")
    from paper_2603_04127_b200 import binding
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    B, H, N, d, r, m, dv = wl.dims()
    # every rank draws its own batch (weak scaling: the workload id, which seeds the data, is shifted by the rank);
    # the parameters M and W are replicated: every rank takes rank 0's
    t = inputs.generate(sharding.rank_workload(wl, rank))
    t.M, t.W = inputs.parameters(wl)
    dt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32

    def host(a):
        return torch.from_numpy(np.ascontiguousarray(a)).to(dt).pin_memory()

    hQ, hK, hV, hM, hW = (host(x) for x in (t.Q, t.K, t.V, t.M, t.W))
    hG = host(t.dO) if wl.backward else None
    Q, K, V, M, W = (x.cuda() for x in (hQ, hK, hV, hM, hW))
    G = hG.cuda() if wl.backward else None
    O = torch.empty_like(V)
    dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
    dM = torch.empty(M.shape, dtype=torch.float32, device="cuda")
    hO, hdQ, hdK, hdV = (torch.empty_like(x).pin_memory() for x in (hV, hQ, hK, hV))
    hdM = torch.empty(M.shape, dtype=torch.float32).pin_memory()

    plan = binding.darkattn_plan(B, H, N, d, m, r=r, dv=dv, dtype=binding.BF16 if wl.dtype == "bf16" else binding.F32,
                                 causal=wl.causal, path=args.path)
    ws = plan.alloc_workspace()
    saved = torch.empty(plan.saved_bytes, dtype=torch.uint8, device="cuda") if plan.saved_bytes else None
    stream = torch.cuda.current_stream()

    def step():
        binding.darkattn_forward(plan, Q, K, V, M, W, O, ws, saved=saved, stream=stream)
        if wl.backward:
            binding.darkattn_backward(plan, Q, K, V, M, W, O, G, dQ, dK, dV, dM, ws, saved=saved, stream=stream)
            sharding.all_reduce_dm(dM)

    # End to end: every step copies its inputs from pinned host memory, runs, and copies its results back. Two sets
    # of device buffers and three streams (upload, compute, download) let the upload of step i+1 and the download of
    # step i-1 run beside the kernels of step i; the copies of one direction and the compute stay in step order.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    sets = []
    for _ in range(2):
        ins = [torch.empty_like(x) for x in (Q, K, V, M, W)] + ([torch.empty_like(G)] if wl.backward else [])
        outs = [torch.empty_like(O)] + ([torch.empty_like(x) for x in (dQ, dK, dV, dM)] if wl.backward else [])
        sets.append({"in": ins, "out": outs, "uploaded": torch.cuda.Event(), "computed": torch.cuda.Event(),
                     "downloaded": torch.cuda.Event()})
    h_in = [hQ, hK, hV, hM, hW] + ([hG] if wl.backward else [])
    h_out = [hO] + ([hdQ, hdK, hdV, hdM] if wl.backward else [])
    e2e_count = [0]

    def e2e_step():
        st = sets[e2e_count[0] % 2]
        reuse = e2e_count[0] >= 2
        e2e_count[0] += 1
        with torch.cuda.stream(s_in):
            if reuse:
                s_in.wait_event(st["computed"])          # the kernels that read this set's inputs are done
            for dst, src in zip(st["in"], h_in):
                dst.copy_(src, non_blocking=True)
            st["uploaded"].record(s_in)
        stream.wait_event(st["uploaded"])
        if reuse:
            stream.wait_event(st["downloaded"])          # this set's previous results have left the device
        q, k, v, mm, ww = st["in"][:5]
        o = st["out"][0]
        binding.darkattn_forward(plan, q, k, v, mm, ww, o, ws, saved=saved, stream=stream)
        if wl.backward:
            g = st["in"][5]
            dq, dk, dv_, dm_ = st["out"][1:]
            binding.darkattn_backward(plan, q, k, v, mm, ww, o, g, dq, dk, dv_, dm_, ws, saved=saved, stream=stream)
            sharding.all_reduce_dm(dm_)
        st["computed"].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(st["computed"])
            for dst, src in zip(h_out, st["out"]):
                dst.copy_(src, non_blocking=True)
            st["downloaded"].record(s_out)

    def e2e_join():
        stream.wait_stream(s_in)
        stream.wait_stream(s_out)

    def timed(fn, steps):
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        return sharding.max_over_ranks(e0.elapsed_time(e1), device="cuda")

    def timed_repeated(fn, steps, min_seconds):
        """Times exactly `steps` steps, again and again until `min_seconds` of device time have been measured (the number
        of repetitions is fixed from the first one, the same on every rank); returns the mean ms of one K-step region,
        the repetitions and all region times."""
        first = timed(fn, steps)
        reps = max(1, int(math.ceil(min_seconds * 1e3 / max(first, 1e-3))))
        regions = [first] + [timed(fn, steps) for _ in range(reps - 1)]
        return float(np.mean(regions)), reps, regions

    for _ in range(args.warmup):
        step()
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(local).uuid).replace("GPU-", ""))
    if rank == 0:
        sampler.start()
    ms, reps, regions = timed_repeated(step, args.steps, args.min_seconds)
    clocks = sampler.stop() if rank == 0 else None
    fwd_ms = timed(lambda: binding.darkattn_forward(plan, Q, K, V, M, W, O, ws, stream=stream), args.steps) / args.steps
    e2e_steps = max(4, min(args.steps, 10))
    e2e_step(); e2e_step(); e2e_join()

    def e2e_run():
        e2e_step()
        if e2e_count[0] == 2 + e2e_steps:                # last timed step: the closing event waits for the copy streams
            e2e_join()

    e2e_ms = timed(e2e_run, e2e_steps) / e2e_steps
    assert binding.darkattn_last_device_status(plan, ws) == binding.OK

    # per-kernel device times: a second pass over the same steps with an event in front of every kernel
    ktimes = {}
    if plan.path == binding.PATH_TENSOR and not args.no_kernel_times:
        binding.darkattn_kernel_timing(plan, True)
        ksteps = args.steps * reps
        for _ in range(ksteps):
            step()
            ktimes = binding.darkattn_kernel_times(plan)
        binding.darkattn_kernel_timing(plan, False)

    ms_step = ms / args.steps
    tokens = B * N
    value = sharding.job_throughput(tokens, world, ms_step * 1e-3)
    h2d = sum(x.numel() * x.element_size() for x in (hQ, hK, hV, hM, hW) + ((hG,) if wl.backward else ()))
    d2h = hO.numel() * hO.element_size() + (sum(x.numel() * x.element_size() for x in (hdQ, hdK, hdV, hdM)) if wl.backward else 0)

    peaks = measured_peaks()
    # the tensor-pipe denominator: the burst figure when the timed region ran at the top SM clock with no power cap (a
    # kernel timed alone), the sustained one otherwise
    at_max = bool(clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and clocks["sm_mhz"] >= 0.97 * clocks["sm_max_mhz"]
                  and "sw_power_cap" not in clocks.get("reasons", []))
    tensor_peak = peaks["bf16_tflops"] if at_max else peaks["bf16_tflops_sustained"]
    tensor_peak_kind = "burst bf16 GEMM (SM clock at its maximum, no power cap during the timed region)" if at_max else "sustained bf16 GEMM"
    th = B * H * N
    flops = flops_per_token_head(d, r, m, dv, 128, wl.causal, wl.backward) * th
    nbytes = bytes_per_token_head(d, dv, wl.backward) * th
    nexp = exps_per_token_head(m, wl.causal, wl.backward) * th
    # cycles per 128x128x16 MMA with both operands in shared memory, alone and beside busy epilogue warps, and the
    # fixed cycles a batch pays between its first issue and the arrival of its commit
    mma_alone, mma_fixed = binding.darkattn_measure_mma_cycles(0, False)
    mma_busy, _ = binding.darkattn_measure_mma_cycles(2, True)
    ex2_peak = binding.darkattn_measure_alu_peak(0, 10)
    fma_peak = binding.darkattn_measure_alu_peak(1, 10)
    legs = {"tensor_us": flops / (tensor_peak * 1e12) * 1e6,
            "exp_us": nexp / ex2_peak * 1e6, "hbm_us": nbytes / (peaks["hbm_gbs"] * 1e9) * 1e6}
    achieved_tf = flops / (ms_step * 1e-3) / 1e12
    whole = {"bound": "tensor", "achieved": achieved_tf, "peak": tensor_peak, "unit": "TFLOP/s",
             "frac": achieved_tf / tensor_peak, "legs_us": legs}
    # each kernel against the slowest of its three legs (tensor at the measured peak chosen above, ex2 at the
    # measured MUFU rate, bytes at the measured copy bandwidth)
    nslab = max(1, m // 128)
    work = kernel_work(d, r, m, dv, 128, nslab, wl.causal)
    kernels = []
    for name, (tot_ms, cnt) in sorted(ktimes.items(), key=lambda kv: -kv[1][0]):
        entry = {"kernel": name, "launches_per_step": cnt / ksteps, "us_per_launch": 1e3 * tot_ms / max(cnt, 1),
                 "us_per_step": 1e3 * tot_ms / ksteps}
        if name in work:
            f, x, b, bound = work[name]
            us = entry["us_per_launch"]
            t_tensor = f * th / (tensor_peak * 1e12) * 1e6
            t_exp = x * th / ex2_peak * 1e6
            t_hbm = b * th / (peaks["hbm_gbs"] * 1e9) * 1e6
            entry.update(bound=bound, legs_us={"tensor_us": t_tensor, "exp_us": t_exp, "hbm_us": t_hbm},
                         frac_of_slowest_leg=max(t_tensor, t_exp, t_hbm) / us)
            if bound == "tensor":
                entry.update(achieved=f * th / (us * 1e-6) / 1e12, unit="TFLOP/s", peak=tensor_peak)
            else:
                entry.update(achieved=b * th / (us * 1e-6) / 1e9, unit="GB/s", peak=peaks["hbm_gbs"])
            entry["frac"] = entry["achieved"] / entry["peak"]
        kernels.append(entry)
    top = next((k for k in kernels if "frac" in k), None)
    traffic = None
    ncu_traffic = ncu_traffic_per_token_head()
    if top is not None and (d, dv, m) == (128, 128, 256) and top["kernel"] in ncu_traffic:
        traffic = ncu_traffic[top["kernel"]] * th
    if top is not None:
        roofline = {"bound": top["bound"], "achieved": top["achieved"], "peak": top["peak"], "unit": top["unit"],
                    "frac": top["frac"], "traffic": traffic, "kernel": top["kernel"],
                    "us_per_launch": top["us_per_launch"], "legs_us": top["legs_us"]}
    else:
        roofline = dict(whole, traffic=None, kernel="whole step")
    sm_mhz = clocks.get("sm_mhz") if clocks else None
    roofline.update(peak_source=peaks["source"] + ": " + tensor_peak_kind + " / copy bandwidth", whole_step=whole, kernels=kernels,
                    ms_per_step_times_sm_mhz=(ms_step * sm_mhz if sm_mhz else None),
                    ex2_per_s_measured=ex2_peak, fma_per_s_measured=fma_peak, forward_ms=fwd_ms,
                    mma_cycles={"ss_alone": mma_alone, "ss_mn_beside_epilogue": mma_busy, "per_batch_fixed": mma_fixed},
                    forward_tokens_per_s=world * tokens / (fwd_ms * 1e-3))

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype,
        "data": "synthetic", "config": {**workload_config(wl), "path": {1: "simt", 2: "tensor"}[plan.path]},
        "clocks": clocks,
        "e2e": {"value": world * tokens / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h},
        "gpu_launches": args.steps * reps * (plan.launches(False) + (plan.launches(True) if wl.backward else 0)),
        "consistency": {"timed_region_s": sum(regions) * 1e-3, "repeats_of_the_k_steps": reps,
                        "ms_per_step_min": min(regions) / args.steps, "ms_per_step_max": max(regions) / args.steps},
        "roofline": roofline,
    }
    if rank == 0 and world == 1 and not args.no_extra_configs:
        del Q, K, V, G, O, dQ, dK, dV, ws, saved, sets
        torch.cuda.empty_cache()
        roofline["configs"] = extra_configs(torch, binding, inputs, peaks, tensor_peak, exclude=args.workload)
        roofline["decode_step"] = decode_benchmark(torch, binding, inputs, peaks)
        roofline["decode_step_large_batch"] = decode_benchmark(torch, binding, inputs, peaks, B=64)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import ref
        sub, use, cores = oracle_sample(wl, inputs, ref)
        t0 = time.perf_counter()
        reps = 2
        for _ in range(reps):
            oracle_step(ref, sub, wl)
        dtc = (time.perf_counter() - t0) / reps
        out["cpu_baseline"] = {"value": len(use) * N / H / dtc, "unit": UNIT, "cores": cores, "kind": "oracle",
                               "sample": f"{len(use)} of {B * H} (batch, head) pairs at full N={N}, "
                                         f"{'forward+backward' if wl.backward else 'forward'}, float64, {reps} repetitions"}
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
