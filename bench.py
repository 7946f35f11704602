#!/usr/bin/env python
"""Benchmark of the DARK-attention hot path: forward + backward tokens/s at N = 8192 on B200.

One step = one forward and one backward call of the whole hot path (feature maps, chunked causal
scan, dQ/dK/dV/dM) over one batch of the synthetic workload. Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload headline]

N > 1 is launched under torch.distributed.run, one rank per GPU; every rank processes its own batch
(weak scaling) and the per-head gradient of M is all-reduced over NCCL, as in data-parallel training.
`--impl reference` times the float64 CPU oracle on the host cores (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# DRAM bytes (read + write) per (token, head) of the scan kernels at d = dv = 128, m = 256 from their ncu capture on the
# small profiling workload (profiles/scan_kernels_d128_small.md); traffic is proportional to the (token, head) count.
# A kernel that changed since its capture has no entry.
NCU_TRAFFIC_PER_TOKEN_HEAD = {"tc_fwd_causal_kernel": 1469.0, "tc_bwd_q_kernel": 2916.0, "tc_bwd_k_kernel": 2797.0}

METRIC = "DARK-attention fwd+bwd tokens/s"
UNIT = "tokens/s"


def flops_per_token_head(d, r, m, dv, C, causal, backward):
    """Algorithmic floating-point operations per (token, head); intra-chunk terms count the lower
    triangle only. Backward: the features are computed once more (query-side kernel; the key-side
    kernel reads them back), and the state before each chunk comes from the forward stash instead of
    being recomputed, so the state terms are dO S^T, R += A^T dO, V R^T and Bf R: 8 m dv."""
    feat = 2 * (2 * d * r + 2 * r * m)                 # both sides: x~ = M x and u = W x~
    fwd = feat + 4 * m * dv + ((C + 1) * (m + dv) if causal else 0)
    if not backward:
        return fwd
    bwd = feat + 8 * m * dv + ((C + 1) * (3 * m + 2 * dv) if causal else 0) + 4 * m * r + 8 * r * d
    return fwd + bwd


def bytes_per_token_head(d, dv, backward, e=2):
    fwd = (2 * d + 2 * dv) * e                          # Q, K, V in; O out
    return fwd + ((4 * d + 4 * dv) * e if backward else 0)   # + Q,K,V,dO in; dQ,dK,dV out (+O)


def exps_per_token_head(m, backward):
    return 2 * m * (2 if backward else 1)


def kernel_work(d, r, m, dv, C, nslab, causal):
    """Algorithmic work per (token, head) of each kernel of the tensor-core path: (flops, exps, bytes,
    bound). The scan kernels split the step's total of flops_per_token_head() between them: the causal
    query-side backward kernel is charged the whole feature recompute (the key-side kernel reads its
    feature tiles back), each backward kernel half of the feature-map backward; bytes count what the
    kernel has to move once (inputs, outputs, and the stashed tiles it reads or writes). The helper
    kernels are HBM-bound and are charged the tensors they read and write once."""
    feat = 2 * (2 * d * r + 2 * r * m)
    tri = C + 1
    e = 2
    k = {
        "tc_fwd_causal_kernel": (feat + 4 * m * dv + tri * (m + dv), 2 * m, (2 * d + 2 * dv) * e, "tensor"),
        "tc_fwd_keys_kernel": (feat // 2 + 2 * m * dv, m, (d + dv) * e, "tensor"),
        "tc_fwd_queries_kernel": (feat // 2 + 2 * m * dv, m, (d + dv) * e, "tensor"),
        "tc_bwd_q_kernel": (feat + 2 * m * dv + tri * (m + dv) + 2 * m * r + 4 * r * d, 2 * m,
                            (3 * d + 2 * dv + 2 * m) * e + m * dv * e // C, "tensor"),
        "tc_bwd_k_kernel": (6 * m * dv + tri * (2 * m + dv) + 2 * m * r + 4 * r * d, 0, (2 * d + 3 * dv + 2 * m) * e, "tensor"),
        "tc_bwd_nc_q_kernel": (feat // 2 + 4 * m * dv + 2 * m * r + 4 * r * d, m, (2 * d + dv) * e, "tensor"),
        "tc_bwd_nc_k_kernel": (feat // 2 + 4 * m * dv + 2 * m * r + 4 * r * d, m, (2 * d + 2 * dv) * e, "tensor"),
        "tc_bwd_finish_k_kernel": (6 * r * d, 0, 3 * d * e, "hbm"),
        "tc_key_norms_kernel": (2 * r * d, 0, d * e + 4, "hbm"),
        "combine_kernel": (0, 0, (nslab * dv + dv) * e + nslab * 8, "hbm"),
        "delta_kernel": (0, 0, 2 * dv * e + 4, "hbm"),
    }
    return k


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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="headline")
    ap.add_argument("--path", type=int, default=0, help="0 auto, 1 SIMT, 2 tensor")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernel-times", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2603_04127_b200 import inputs
    wl = inputs.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
        return

    import torch
    import torch.distributed as dist
    from paper_2603_04127_b200 import binding

    from paper_2603_04127_b200 import sharding
    rank, world, local = sharding.env_rank_world()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    B, H, N, d, r, m, dv = wl.dims()
    # every rank draws its own batch (weak scaling): shift the workload id by the rank
    t = inputs.generate(sharding.rank_workload(wl, rank))
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

    for _ in range(args.warmup):
        step()
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(local).uuid).replace("GPU-", ""))
    if rank == 0:
        sampler.start()
    ms = timed(step, args.steps)
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
        for _ in range(args.steps):
            step()
            ktimes = binding.darkattn_kernel_times(plan)
        binding.darkattn_kernel_timing(plan, False)

    ms_step = ms / args.steps
    tokens = B * N
    value = sharding.job_throughput(tokens, world, ms_step * 1e-3)
    h2d = sum(x.numel() * x.element_size() for x in (hQ, hK, hV, hM, hW) + ((hG,) if wl.backward else ()))
    d2h = hO.numel() * hO.element_size() + (sum(x.numel() * x.element_size() for x in (hdQ, hdK, hdV, hdM)) if wl.backward else 0)

    peaks = measured_peaks()
    th = B * H * N
    flops = flops_per_token_head(d, r, m, dv, 128, wl.causal, wl.backward) * th
    nbytes = bytes_per_token_head(d, dv, wl.backward) * th
    nexp = exps_per_token_head(m, wl.backward) * th
    # cycles per 128x128x16 MMA with both operands in shared memory, alone and beside busy epilogue warps, and the
    # fixed cycles a batch pays between its first issue and the arrival of its commit
    mma_alone, mma_fixed = binding.darkattn_measure_mma_cycles(0, False)
    mma_busy, _ = binding.darkattn_measure_mma_cycles(2, True)
    ex2_peak = binding.darkattn_measure_alu_peak(0, 10)
    fma_peak = binding.darkattn_measure_alu_peak(1, 10)
    legs = {"tensor_us": flops / (peaks["bf16_tflops_sustained"] * 1e12) * 1e6,
            "exp_us": nexp / ex2_peak * 1e6, "hbm_us": nbytes / (peaks["hbm_gbs"] * 1e9) * 1e6}
    achieved_tf = flops / (ms_step * 1e-3) / 1e12
    whole = {"bound": "tensor", "achieved": achieved_tf, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
             "frac": achieved_tf / peaks["bf16_tflops_sustained"], "legs_us": legs}
    # each kernel against the slowest of its three legs (tensor at the sustained measured peak, ex2 at the
    # measured MUFU rate, bytes at the measured copy bandwidth)
    nslab = max(1, m // 128)
    work = kernel_work(d, r, m, dv, 128, nslab, wl.causal)
    kernels = []
    for name, (tot_ms, cnt) in sorted(ktimes.items(), key=lambda kv: -kv[1][0]):
        entry = {"kernel": name, "launches_per_step": cnt / args.steps, "us_per_launch": 1e3 * tot_ms / max(cnt, 1),
                 "us_per_step": 1e3 * tot_ms / args.steps}
        if name in work:
            f, x, b, bound = work[name]
            us = entry["us_per_launch"]
            t_tensor = f * th / (peaks["bf16_tflops_sustained"] * 1e12) * 1e6
            t_exp = x * th / ex2_peak * 1e6
            t_hbm = b * th / (peaks["hbm_gbs"] * 1e9) * 1e6
            entry.update(bound=bound, legs_us={"tensor_us": t_tensor, "exp_us": t_exp, "hbm_us": t_hbm},
                         frac_of_slowest_leg=max(t_tensor, t_exp, t_hbm) / us)
            if bound == "tensor":
                entry.update(achieved=f * th / (us * 1e-6) / 1e12, unit="TFLOP/s", peak=peaks["bf16_tflops_sustained"])
            else:
                entry.update(achieved=b * th / (us * 1e-6) / 1e9, unit="GB/s", peak=peaks["hbm_gbs"])
            entry["frac"] = entry["achieved"] / entry["peak"]
        kernels.append(entry)
    top = next((k for k in kernels if "frac" in k), None)
    traffic = None
    if top is not None and (d, dv, m) == (128, 128, 256) and top["kernel"] in NCU_TRAFFIC_PER_TOKEN_HEAD:
        traffic = NCU_TRAFFIC_PER_TOKEN_HEAD[top["kernel"]] * th
    if top is not None:
        roofline = {"bound": top["bound"], "achieved": top["achieved"], "peak": top["peak"], "unit": top["unit"],
                    "frac": top["frac"], "traffic": traffic, "kernel": top["kernel"],
                    "us_per_launch": top["us_per_launch"], "legs_us": top["legs_us"]}
    else:
        roofline = dict(whole, traffic=None, kernel="whole step")
    roofline.update(peak_source=peaks["source"] + " (sustained bf16 GEMM / copy bandwidth)", whole_step=whole, kernels=kernels,
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
        "gpu_launches": args.steps * (plan.launches(False) + (plan.launches(True) if wl.backward else 0)),
        "roofline": roofline,
    }
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
