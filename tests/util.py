"""Helpers of the GPU parity tests: move a synthetic workload to the device, run the library through
its C ABI, and compare with the float64 oracle."""
from __future__ import annotations

import numpy as np
import torch

from paper_2603_04127_b200 import inputs

TOL = {"f32": 1e-4, "bf16": 2e-2}   # relative error bars (Frobenius-relative and max-relative)


def to_dev(a, dtype):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to("cuda").to(dtype).contiguous()


def torch_dtype(name):
    return torch.float32 if name == "f32" else torch.bfloat16


def run_gpu(binding, wl, t, path=0, chunk=0, scale=0.0, backward=None, w_per_head=False, use_saved=False, want_dw=False):
    """Run forward (and backward) on the device for tensors ``t`` laid out [B', H', N, *].

    With ``use_saved`` the forward call fills the plan's forward->backward stash and the backward call
    is given it (and O); otherwise backward gets neither and recomputes what it needs."""
    Bq, Hq, N, d = t.Q.shape
    dv = t.V.shape[-1]
    r = t.M.shape[-2]
    m = t.W.shape[-2]
    dt = torch_dtype(wl.dtype)
    Hkv = t.K.shape[1]                                    # fewer key/value heads than query heads: grouped heads
    plan = binding.darkattn_plan(Bq, Hq, N, d, m, r=r, dv=dv, dtype=binding.F32 if wl.dtype == "f32" else binding.BF16,
                                 causal=wl.causal, chunk=chunk, scale=scale, w_per_head=w_per_head, path=path,
                                 H_kv=0 if Hkv == Hq else Hkv)
    ws = plan.alloc_workspace()
    Q, K, V, M, W = (to_dev(x, dt) for x in (t.Q, t.K, t.V, t.M, t.W))
    O = torch.empty((Bq, Hq, N, dv), dtype=dt, device="cuda")     # (V may have fewer heads: grouped key/value heads)
    saved = None
    if use_saved and plan.saved_bytes:
        saved = torch.empty(plan.saved_bytes, dtype=torch.uint8, device="cuda")
    binding.darkattn_forward(plan, Q, K, V, M, W, O, ws, saved=saved)
    out = {"O": O.float().cpu().numpy().astype(np.float64)}
    do_bwd = wl.backward if backward is None else backward
    if do_bwd:
        dO = to_dev(t.dO, dt)
        dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
        dM = torch.empty(M.shape, dtype=torch.float32, device="cuda")
        binding.darkattn_backward(plan, Q, K, V, M, W, O if saved is not None else None, dO, dQ, dK, dV, dM, ws,
                                  saved=saved)
        for k, v in (("dQ", dQ), ("dK", dK), ("dV", dV), ("dM", dM)):
            out[k] = v.float().cpu().numpy().astype(np.float64)
        if want_dw:
            dW = torch.empty(W.shape, dtype=torch.float32, device="cuda")
            binding.darkattn_backward_dw(plan, M, dW, ws)
            out["dW"] = dW.cpu().numpy().astype(np.float64)
    assert binding.darkattn_last_device_status(plan, ws) == binding.OK
    torch.cuda.synchronize()
    plan.destroy()
    return out


def rel_errors(got, want):
    fro = np.linalg.norm((got - want).ravel()) / max(np.linalg.norm(want.ravel()), 1e-300)
    mx = np.abs(got - want).max() / max(np.abs(want).max(), 1e-300)
    return fro, mx


def assert_close(got, want, tol, what):
    assert np.isfinite(got).all(), f"{what}: non-finite values"
    fro, mx = rel_errors(got, want)
    assert fro < tol and mx < tol, f"{what}: frobenius-relative {fro:.3e}, max-relative {mx:.3e} (bar {tol:g})"
    return fro, mx
