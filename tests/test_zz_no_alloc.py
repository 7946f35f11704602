"""darkattn_forward_static: the forward pass for hosts that cannot allocate device memory.

A serving process that handed the whole GPU to its own memory pool, or a plug-in that only ever sees
input and output buffers, has no workspace to give and must not call cudaMalloc. The static entry
point keeps its intermediates in an array inside the library instead. These tests call it through
the C ABI and hold it to the ordinary entry point's result and to the float64 oracle, twice in a row
because the array keeps the previous call's contents. The file sorts last on purpose, so a run that stops at the first
failure has already been through every other test.
"""
import numpy as np
import pytest
import torch

from paper_2603_04127_b200 import inputs
from tests.util import TOL, rel_errors, to_dev, torch_dtype


@pytest.fixture(scope="module")
def binding():
    from paper_2603_04127_b200 import build
    build.build()
    from paper_2603_04127_b200 import binding as b
    return b


def _have_library():
    import os
    import shutil
    here = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    return os.path.exists(os.path.join(here, "paper_2603_04127_b200", "libdarkattn.so")) or shutil.which("nvcc") or os.path.exists("/usr/local/cuda/bin/nvcc")


@pytest.mark.skipif(not _have_library(), reason="neither libdarkattn.so nor nvcc to build it")
def test_oversized_problem_is_refused_on_the_host(binding):
    plan = binding.darkattn_plan(4, 16, 8192, 128, 256, dtype=binding.BF16, causal=True)
    assert binding.darkattn_static_scratch_needed(plan) > binding.STATIC_SCRATCH_BYTES
    a = 4096  # never dereferenced: the size check comes before any GPU work
    rc = binding.lib.darkattn_forward_static(plan.handle, a, a, a, a, a, a, None)
    assert rc == binding.ERR_WORKSPACE
    plan.destroy()


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,causal", [("f32", False), ("bf16", True)])
def test_static_scratch_forward_matches_workspace_forward(binding, dtype, causal):
    wl = inputs.small(name="noalloc", wid=41, B=1, H=2, N=300, d=64, m=128, dtype=dtype, causal=causal,
                      backward=False)
    t = inputs.generate(wl)
    dt = torch_dtype(dtype)
    Q, K, V, M, W = (to_dev(x, dt) for x in (t.Q, t.K, t.V, t.M, t.W))
    plan = binding.darkattn_plan(1, 2, 300, 64, 128, dtype=binding.F32 if dtype == "f32" else binding.BF16,
                                 causal=causal, path=binding.PATH_SIMT)
    assert 0 < binding.darkattn_static_scratch_needed(plan) <= binding.STATIC_SCRATCH_BYTES
    ws = plan.alloc_workspace()
    want = torch.empty_like(V)
    binding.darkattn_forward(plan, Q, K, V, M, W, want, ws)
    torch.cuda.synchronize()
    want = want.float().cpu().numpy()
    from oracle import ref
    exact = ref.forward(t.Q, t.K, t.V, t.M, t.W, causal=causal)
    for call in range(2):
        # the second call runs on a different problem's leftovers: swap queries and keys in between
        if call == 1:
            junk = torch.empty_like(V)
            binding.darkattn_forward_static(plan, K, Q, V, M, W, junk)
        got = torch.full_like(V, float("nan"))
        binding.darkattn_forward_static(plan, Q, K, V, M, W, got)
        torch.cuda.synchronize()
        got = got.float().cpu().numpy()
        assert np.isfinite(got).all()
        fro, mx = rel_errors(got.astype(np.float64), want.astype(np.float64))
        assert fro < TOL[dtype] and mx < TOL[dtype], (call, fro, mx)
        fro, mx = rel_errors(got.astype(np.float64), exact)          # and against the oracle, like every other entry point
        assert fro < TOL[dtype] and mx < TOL[dtype], ("oracle", call, fro, mx)
    plan.destroy()
