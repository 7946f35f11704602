"""Element-wise parity of the CUDA path (through the C ABI) with the float64 oracle."""
import numpy as np
import pytest

from oracle import ref
from paper_2603_04127_b200 import inputs
from tests.util import TOL, assert_close, run_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2603_04127_b200 import binding as b
    return b


def _oracle(t, wl, scale=None, backward=None):
    out = {"O": ref.forward(t.Q, t.K, t.V, t.M, t.W, causal=wl.causal, scale=scale)}
    if wl.backward if backward is None else backward:
        dQ, dK, dV, dM, _ = ref.backward(t.Q, t.K, t.V, t.M, t.W, t.dO, causal=wl.causal, scale=scale)
        out.update(dQ=dQ, dK=dK, dV=dV, dM=dM)
    return out


def _compare(got, want, tol, tag):
    for k in want:
        assert_close(got[k], want[k], tol, f"{tag}:{k}")


def test_c1_fp32_noncausal_forward(binding):
    wl = inputs.WORKLOADS["c1"]
    t = inputs.generate(wl)
    _compare(run_gpu(binding, wl, t), _oracle(t, wl), TOL["f32"], "c1")


SMALL = [
    # name, kwargs: sizes span several 64-wide tiles and ragged tails
    ("nc_ragged", dict(B=2, H=3, N=200, d=48, m=80, causal=False)),
    ("nc_lowrank", dict(B=1, H=2, N=130, d=64, m=96, r=24, dv=40, causal=False)),
    ("causal_ragged", dict(B=2, H=2, N=333, d=32, m=72, causal=True)),
    ("causal_lowrank", dict(B=1, H=3, N=257, d=64, m=64, r=16, dv=72, causal=True)),
    ("one_token", dict(B=1, H=1, N=1, d=8, m=8, causal=True)),
    ("one_chunk", dict(B=1, H=2, N=128, d=64, m=128, causal=True)),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("name,kw", SMALL, ids=[s[0] for s in SMALL])
def test_small_shapes_forward_backward_simt(binding, name, kw, dtype):
    wl = inputs.small(name=name, wid=20 + len(name), dtype=dtype, backward=True, **kw)
    t = inputs.generate(wl)
    got = run_gpu(binding, wl, t, path=binding.PATH_SIMT)
    want = _oracle(t, wl)
    if name == "one_token":
        # O_0 = V_0 whatever Q, K and M are: those gradients are exactly zero, so compare them absolutely
        for k in ("dQ", "dK", "dM"):
            assert np.abs(want.pop(k)).max() < 1e-12 and np.abs(got[k]).max() < TOL[dtype]
    _compare(got, want, TOL[dtype], name)


@pytest.mark.parametrize("chunk", [16, 64, 256])
def test_chunk_length_does_not_change_the_result(binding, chunk):
    wl = inputs.small(name="chunks", wid=31, B=1, H=2, N=300, d=32, m=64, causal=True, dtype="f32")
    t = inputs.generate(wl)
    _compare(run_gpu(binding, wl, t, chunk=chunk), _oracle(t, wl), TOL["f32"], f"chunk{chunk}")


def test_explicit_scale_and_per_head_projections(binding):
    wl = inputs.small(name="wph", wid=32, B=2, H=2, N=96, d=16, m=32, causal=True, dtype="f32")
    t = inputs.generate(wl)
    rng = np.random.default_rng(5)
    t.W = rng.standard_normal((2, 32, 16)).astype(np.float32).astype(np.float64)
    got = run_gpu(binding, wl, t, scale=0.2, w_per_head=True)
    _compare(got, _oracle(t, wl, scale=0.2), TOL["f32"], "wph")


@pytest.mark.parametrize("case", ["simt_f32", "tensor_bf16_causal", "tensor_bf16_noncausal"])
def test_large_norm_inputs_stay_finite(binding, case):
    """Queries and keys six times larger: exponents far outside exp's fp32 range without the stabilising shifts, which
    are taken from the data on both paths (row maxima for the queries, the maximum over the keys for the key features)."""
    if case == "simt_f32":
        wl = inputs.small(name="bignorm", wid=33, B=1, H=1, N=192, d=32, m=64, causal=False, dtype="f32", backward=False)
        path, tol = binding.PATH_SIMT, 5e-4     # the exponent's argument is ~36 times larger, and so is its fp32 rounding
    else:
        wl = inputs.small(name="bignorm", wid=33, B=1, H=2, N=384, d=64, m=256, causal="noncausal" not in case, dtype="bf16",
                          backward=True)
        path, tol = binding.PATH_TENSOR, TOL["bf16"]
    t = inputs.generate(wl)
    # a causal prefix sees only some of the keys while the key-side shift is one constant per (batch, head, slab): the
    # spread of the exponents between prefixes, which grows with the square of the scale, has to stay within fp32's range
    scale = 4.0 if case == "tensor_bf16_causal" else 6.0
    t.Q = t.Q * scale
    t.K = t.K * scale
    if wl.dtype == "bf16":
        t.Q, t.K = (inputs.round_to_bf16(x).astype(np.float64) for x in (t.Q, t.K))
    got = run_gpu(binding, wl, t, path=path, use_saved=True)
    _compare(got, _oracle(t, wl), tol, case)


FULL = {
    # workload -> (b, h) pairs checked against the oracle at full sequence length
    "c2": [(0, 0), (3, 7), (7, 11)],
    "c3": [(0, 0), (3, 15)],
    "c4": [(0, 0), (0, 7)],
}


@pytest.mark.parametrize("name", list(FULL))
def test_full_size_forward_sampled_heads(binding, name):
    wl = inputs.WORKLOADS[name]
    t = inputs.generate(wl)
    got = run_gpu(binding, wl, t)["O"]
    sub = inputs.generate(wl, pairs=FULL[name])
    want = _oracle(sub, wl)["O"]
    for i, (b, h) in enumerate(FULL[name]):
        assert_close(got[b, h], want[0, i], TOL[wl.dtype], f"{name}[{b},{h}]")


def test_c5_training_step(binding):
    wl = inputs.WORKLOADS["c5"]
    B, H = wl.B, wl.H
    t = inputs.generate(wl)
    got = run_gpu(binding, wl, t)
    # the gradient of M_h sums over the batch: check two heads over every batch entry
    for h in (0, H - 1):
        pairs = [(b, h) for b in range(B)]
        sub = inputs.generate(wl, pairs=pairs, as_batch=True)
        want = _oracle(sub, wl)   # B' = B pairs, H' = 1, so dM sums over them
        for k in ("O", "dQ", "dK", "dV"):
            g = np.stack([got[k][b, h] for b in range(B)])[:, None]
            assert_close(g, want[k], TOL["bf16"], f"c5 head {h}: {k}")
        assert_close(got["dM"][h], want["dM"][0], TOL["bf16"], f"c5 head {h}: dM")


TENSOR = [
    # shapes the tcgen05 kernels cover: d, dv in {64,128}; m, N multiples of 128
    ("nc_d64_m128", dict(B=1, H=2, N=256, d=64, m=128, causal=False)),
    ("nc_d64_m256", dict(B=2, H=3, N=640, d=64, m=256, causal=False)),
    ("nc_d128_m256", dict(B=1, H=2, N=384, d=128, m=256, causal=False)),
    ("nc_d64_dv128_r32", dict(B=1, H=2, N=256, d=64, m=128, dv=128, r=32, causal=False)),
    ("c_one_chunk", dict(B=1, H=1, N=128, d=64, m=128, causal=True)),
    ("c_d64_m128", dict(B=1, H=2, N=512, d=64, m=128, causal=True)),
    ("c_d64_m512", dict(B=2, H=2, N=384, d=64, m=512, causal=True)),
    ("c_d128_m256", dict(B=1, H=3, N=640, d=128, m=256, causal=True)),
    ("c_d128_dv64_r64", dict(B=1, H=2, N=256, d=128, m=128, dv=64, r=64, causal=True)),
    # few long sequences: the causal scan is cut into segments that run side by side
    ("c_segmented_d64", dict(B=1, H=2, N=2048, d=64, m=256, causal=True)),
    ("c_segmented_d128", dict(B=1, H=1, N=1536, d=128, m=128, dv=64, causal=True)),
]


@pytest.mark.parametrize("name,kw", TENSOR, ids=[s[0] for s in TENSOR])
def test_tensor_path_forward(binding, name, kw):
    wl = inputs.small(name=name, wid=50 + len(name), dtype="bf16", backward=False, **kw)
    t = inputs.generate(wl)
    got = run_gpu(binding, wl, t, path=binding.PATH_TENSOR)
    _compare(got, _oracle(t, wl), TOL["bf16"], name)


TENSOR_BWD = [
    ("b_one_chunk", dict(B=1, H=1, N=128, d=64, m=128, causal=True)),
    ("b_d64_m128", dict(B=1, H=2, N=512, d=64, m=128, causal=True)),
    ("b_d64_m512", dict(B=2, H=2, N=384, d=64, m=512, causal=True)),
    ("b_d128_m256", dict(B=2, H=3, N=640, d=128, m=256, causal=True)),
    ("b_d128_dv64_r64", dict(B=1, H=2, N=256, d=128, m=128, dv=64, r=64, causal=True)),
    ("b_d64_dv128_r32", dict(B=2, H=2, N=384, d=64, m=256, dv=128, r=32, causal=True)),
    ("b_segmented_fwd", dict(B=1, H=2, N=1024, d=64, m=128, causal=True)),
    # eight slabs of features (the general-slab-count code paths), smallest projection rank
    ("b_m1024_r16", dict(B=1, H=2, N=256, d=64, m=1024, r=16, causal=True)),
    ("b_nc_m1024", dict(B=1, H=1, N=256, d=64, m=1024, causal=False)),
    # projection ranks that end inside a warp's 32 rows
    ("b_r48", dict(B=1, H=2, N=256, d=64, m=128, r=48, causal=True)),
    ("b_nc_r16_d128", dict(B=1, H=2, N=256, d=128, m=256, r=16, causal=False)),
    # more (batch, head, chunk) items than CTA groups: a query-side CTA walks several runs, across heads
    ("b_m512_runs", dict(B=2, H=4, N=2048, d=64, m=512, causal=True)),
    ("b_d128_dv64_runs", dict(B=2, H=20, N=1024, d=128, m=128, dv=64, causal=True)),
    # no causal mask: one pass over the queries, one over the keys
    ("b_nc_one_tile", dict(B=1, H=1, N=128, d=64, m=128, causal=False)),
    ("b_nc_d64_m256", dict(B=2, H=3, N=640, d=64, m=256, causal=False)),
    ("b_nc_d128_m256", dict(B=1, H=2, N=384, d=128, m=256, causal=False)),
    ("b_nc_d128_dv64_r64", dict(B=1, H=2, N=256, d=128, m=128, dv=64, r=64, causal=False)),
    ("b_nc_d64_dv128_r32", dict(B=2, H=2, N=384, d=64, m=512, dv=128, r=32, causal=False)),
    ("b_nc_pieces", dict(B=1, H=1, N=2048, d=64, m=128, causal=False)),
]


@pytest.mark.parametrize("use_saved", [False, True], ids=["recompute", "saved"])
@pytest.mark.parametrize("name,kw", TENSOR_BWD, ids=[s[0] for s in TENSOR_BWD])
def test_tensor_path_backward(binding, name, kw, use_saved):
    wl = inputs.small(name=name, wid=70 + len(name), dtype="bf16", backward=True, **kw)
    t = inputs.generate(wl)
    got = run_gpu(binding, wl, t, path=binding.PATH_TENSOR, use_saved=use_saved)
    _compare(got, _oracle(t, wl), TOL["bf16"], name)


# Shapes drawn at random over everything the tensor-core path accepts (three and five feature slabs, projection ranks
# that are not multiples of 32 or exceed d, d != dv, per-head projection rows, recompute and stash), kept as a fixed list.
MIXED = [
    dict(B=1, H=1, N=128, d=64, dv=128, m=640, r=16, causal=False, saved=True, wph=False),
    dict(B=2, H=1, N=256, d=128, dv=64, m=384, r=32, causal=False, saved=False, wph=True),
    dict(B=3, H=2, N=384, d=128, dv=128, m=640, r=96, causal=True, saved=False, wph=True),
    dict(B=2, H=1, N=640, d=128, dv=128, m=640, r=48, causal=True, saved=False, wph=False),
    dict(B=2, H=1, N=256, d=64, dv=128, m=256, r=80, causal=True, saved=False, wph=True),
    dict(B=1, H=1, N=256, d=64, dv=128, m=512, r=112, causal=True, saved=False, wph=False),
    dict(B=3, H=3, N=640, d=64, dv=128, m=128, r=80, causal=True, saved=True, wph=False),
    dict(B=1, H=3, N=384, d=128, dv=64, m=256, r=112, causal=False, saved=True, wph=False),
    dict(B=1, H=2, N=3072, d=64, dv=64, m=384, r=128, causal=True, saved=True, wph=False),
    dict(B=1, H=1, N=4096, d=128, dv=64, m=256, r=64, causal=True, saved=False, wph=False),
]


@pytest.mark.parametrize("i", range(len(MIXED)))
def test_tensor_path_mixed_shapes(binding, i):
    kw = dict(MIXED[i])
    saved, wph = kw.pop("saved"), kw.pop("wph")
    wl = inputs.small(name=f"mixed{i}", wid=300 + i, dtype="bf16", backward=True, **kw)
    t = inputs.generate(wl)
    if wph:
        rng = np.random.default_rng(300 + i)
        t.W = inputs.round_to_bf16(rng.standard_normal((wl.H,) + t.W.shape)).astype(np.float64)
    got = run_gpu(binding, wl, t, path=binding.PATH_TENSOR, use_saved=saved, w_per_head=wph)
    _compare(got, _oracle(t, wl), TOL["bf16"], wl.name)


def test_tensor_path_per_head_projections_and_scale(binding):
    wl = inputs.small(name="t_wph", wid=77, B=2, H=3, N=384, d=64, m=256, causal=True, dtype="bf16", backward=True)
    t = inputs.generate(wl)
    rng = np.random.default_rng(11)
    t.W = inputs.round_to_bf16(rng.standard_normal((3, 256, 64))).astype(np.float64)
    got = run_gpu(binding, wl, t, path=binding.PATH_TENSOR, scale=0.2, w_per_head=True, use_saved=True)
    _compare(got, _oracle(t, wl, scale=0.2), TOL["bf16"], "t_wph")


@pytest.mark.parametrize("case", ["simt_f32", "simt_f32_noncausal_wph", "tensor", "tensor_wph", "tensor_noncausal"])
def test_gradient_of_the_projection_rows(binding, case):
    wph = case.endswith("wph")
    tensor = case.startswith("tensor")
    kw = dict(B=2, H=3, N=384, d=64, m=256, causal="noncausal" not in case) if tensor else dict(B=2, H=2, N=150, d=24, m=40, r=16, causal="noncausal" not in case)
    wl = inputs.small(name=case, wid=81, dtype="bf16" if tensor else "f32", backward=True, **kw)
    t = inputs.generate(wl)
    if wph:
        rng = np.random.default_rng(12)
        W = rng.standard_normal((wl.H,) + t.W.shape)
        t.W = inputs.round_to_bf16(W).astype(np.float64) if tensor else W.astype(np.float32).astype(np.float64)
    got = run_gpu(binding, wl, t, path=binding.PATH_TENSOR if tensor else binding.PATH_SIMT, w_per_head=wph, want_dw=True)
    want = ref.backward(t.Q, t.K, t.V, t.M, t.W, t.dO, causal=wl.causal)[4]
    assert_close(got["dW"], want, TOL[wl.dtype], f"{case}: dW")


DECODE = [
    ("few_heads", dict(B=2, H=3, N=40, d=32, m=96, r=16, dv=64)),
    # several thousand (batch, head) pairs: more blocks than one wave of the GPU holds
    ("many_heads_dv128", dict(B=64, H=48, N=5, d=32, m=64, r=16, dv=128)),
    # dv = 96: 512 / 96 = 5 feature groups and 32 idle threads; m = 640 > 512: more than one feature per thread in the
    # normaliser; rows of M (d = 48) are read with 16-byte loads, rows of W (r = 20) are not multiples of 16 bytes and take
    # the element-wise loop
    ("dv96_m640", dict(B=1, H=2, N=12, d=48, m=640, r=20, dv=96)),
    ("dv512", dict(B=1, H=1, N=6, d=64, m=128, r=64, dv=512)),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("name,kw", DECODE, ids=[s[0] for s in DECODE])
def test_decode_steps_reproduce_the_causal_forward(binding, name, kw, dtype):
    """Token by token through the recurrent entry point: step t's output is row t of the causal attention."""
    import torch
    from tests.util import to_dev, torch_dtype
    wl = inputs.small(name="decode_" + name, wid=83, causal=True, dtype=dtype, backward=False, **kw)
    t = inputs.generate(wl)
    dt = torch_dtype(dtype)
    B, H, N, d, m, r, dv = (kw[k] for k in ("B", "H", "N", "d", "m", "r", "dv"))
    Q, K, V, M, W = (to_dev(x, dt) for x in (t.Q, t.K, t.V, t.M, t.W))
    plan = binding.darkattn_plan(B, H, N, d, m, r=r, dv=dv, dtype=binding.F32 if dtype == "f32" else binding.BF16, causal=True)
    S = torch.zeros(B, H, m, dv, dtype=torch.float32, device="cuda")
    z = torch.zeros(B, H, m, dtype=torch.float32, device="cuda")
    rows = []
    for i in range(N):
        o = torch.empty(B, H, dv, dtype=dt, device="cuda")
        binding.darkattn_decode_step(plan, Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous(), M, W, S, z, o)
        rows.append(o.float().cpu().numpy().astype(np.float64))
    got = np.stack(rows, axis=2)
    want = ref.forward(t.Q, t.K, t.V, t.M, t.W, causal=True)
    assert_close(got, want, 1e-4 if dtype == "f32" else 1e-2, f"decode {name} {dtype}")
    plan.destroy()


@pytest.mark.parametrize("name", ["headline", "headline_nc"])
def test_headline_backward_sampled_heads(binding, name):
    """Forward + backward at the benchmark's full size; dQ, dK, dV of sampled (batch, head) pairs and
    the gradient of M of one head (summed over the whole batch) against the oracle."""
    wl = inputs.WORKLOADS[name]
    B, H = wl.B, wl.H
    t = inputs.generate(wl)
    got = run_gpu(binding, wl, t, use_saved=True)
    h = 5
    pairs = [(b, h) for b in range(B)]
    sub = inputs.generate(wl, pairs=pairs, as_batch=True)
    want = _oracle(sub, wl)
    for k in ("O", "dQ", "dK", "dV"):
        g = np.stack([got[k][b, h] for b in range(B)])[:, None]
        assert_close(g, want[k], TOL["bf16"], f"{name} head {h}: {k}")
    assert_close(got["dM"][h], want["dM"][0], TOL["bf16"], f"{name} head {h}: dM")


SWEEP = [(wid, dict(B=2, H=2, N=512, d=64, m=256)) for wid in range(1, 11)] + \
        [(wid, dict(B=1, H=2, N=1024, d=128, m=256)) for wid in (3, 7, 11)]


@pytest.mark.parametrize("causal", [True, False], ids=["causal", "noncausal"])
@pytest.mark.parametrize("wid,kw", SWEEP, ids=[f"id{w}_d{k['d']}" for w, k in SWEEP])
def test_bf16_error_over_many_seeds(binding, wid, kw, causal):
    """The bf16 bar must hold with margin whatever the random draw: ten workload ids at the smoke shape (among them
    id 7, the draw on which one element of dQ once missed the bar) and three at d = 128, forward and backward. Every
    tensor meets the bar in both measures and its Frobenius-relative error stays below 1e-2 (observed: 0.3 to 0.7 %);
    the largest single deviation and the worst element-wise relative error over the elements above 1 % of the maximum
    are printed."""
    wl = inputs.small(name="sweep", wid=wid, dtype="bf16", causal=causal, backward=True, **kw)
    t = inputs.generate(wl)
    got = run_gpu(binding, wl, t, path=binding.PATH_TENSOR, use_saved=True)
    want = _oracle(t, wl)
    for k, w in want.items():
        fro, mx = assert_close(got[k], w, TOL["bf16"], f"sweep id {wid} {k}")
        big = np.abs(w) > 0.01 * np.abs(w).max()
        ew = (np.abs(got[k] - w)[big] / np.abs(w)[big]).max()
        print(f"sweep id {wid} d={kw['d']} causal={int(causal)} {k}: fro {fro:.2e} max {mx:.2e} worst element-wise {ew:.2e}")
        assert fro < 1e-2, (wid, k, fro, mx)


GROUPED = [
    # path, H, H_kv, shape
    ("simt_f32", 4, 1, dict(B=2, N=150, d=24, m=40, r=16, dv=20)),
    ("simt_f32", 6, 3, dict(B=1, N=130, d=16, m=32)),
    ("tensor", 4, 1, dict(B=2, N=384, d=64, m=256)),
    ("tensor", 8, 2, dict(B=1, N=256, d=128, m=128, dv=64)),
    ("tensor", 4, 4, dict(B=1, N=256, d=64, m=128)),
    # four slabs and two query heads per key/value head: eight parts per element of dK and dV. Added straight into the shared
    # bf16 rows they put dK over the bar; each query head's parts go to rows of its own and the group is summed in fp32
    ("tensor", 2, 1, dict(B=2, N=384, d=128, m=512, r=48, dv=128)),
]


@pytest.mark.parametrize("causal", [True, False], ids=["causal", "noncausal"])
@pytest.mark.parametrize("path,H,Hkv,kw", GROUPED, ids=[f"{g[0]}_H{g[1]}_Hkv{g[2]}" for g in GROUPED])
def test_grouped_key_value_heads(binding, path, H, Hkv, kw, causal):
    """K and V with fewer heads than Q (H_kv in {1, H/4 .., H}): query heads h*G .. h*G+G-1 read key/value head h; dK and dV
    sum over the group. Forward and backward against the oracle, on the FP32 and on the tensor-core kernels."""
    dtype = "f32" if path == "simt_f32" else "bf16"
    wl = inputs.small(name="grouped", wid=95, H=H, dtype=dtype, causal=causal, backward=True, **kw)
    t = inputs.generate(wl)
    G = H // Hkv
    t.K, t.V = np.ascontiguousarray(t.K[:, ::G]), np.ascontiguousarray(t.V[:, ::G])     # keep every G-th head as the shared one
    got = run_gpu(binding, wl, t, path=binding.PATH_SIMT if path == "simt_f32" else binding.PATH_TENSOR, use_saved=True)
    want = _oracle(t, wl)
    assert got["dK"].shape == t.K.shape and got["dV"].shape == t.V.shape
    _compare(got, want, TOL[dtype], f"grouped {path} H={H} H_kv={Hkv}")


def test_tensor_path_is_deterministic(binding):
    """The scan kernels hand tiles between warps through shared and tensor memory; a missing wait shows up as rare,
    run-dependent errors of the size of the values themselves. O has a fixed summation order: repeated runs at the
    benchmark's size must agree bit for bit. The gradients contain sums whose order is not fixed (shared-memory and
    global atomics), so repeated runs may differ in the last bf16 bit of an element, but by no more."""
    wl = inputs.WORKLOADS["headline"]
    t = inputs.generate(wl)
    first = run_gpu(binding, wl, t, use_saved=True)
    for _ in range(3):
        again = run_gpu(binding, wl, t, use_saved=True)
        assert np.array_equal(first["O"], again["O"]), "O differs between runs"
        for k in ("dQ", "dK", "dV"):
            worst = np.abs(first[k] - again[k]).max() / np.abs(first[k]).max()
            assert worst < 2.0 ** -7, f"{k} differs between runs by {worst:.2e} of its largest value"


@pytest.mark.parametrize("causal", [False, True], ids=["noncausal", "causal"])
@pytest.mark.parametrize("aligned", [False, True], ids=["isotropic", "aligned"])
def test_variance_workload_on_the_tensor_path(binding, aligned, causal):
    """The second synthetic workload (Gaussian inputs below the Theorem 3.2 bound, orthogonal projection rows, M the
    identity or the variance-optimal geometry, scale 1), forward and backward, against the oracle."""
    t = inputs.variance_workload(wid=23, B=2, H=2, N=512, d=64, m=256, lam_max=0.2, aligned=aligned, causal=causal)
    got = run_gpu(binding, t.wl, t, path=binding.PATH_TENSOR, scale=1.0, use_saved=True)
    _compare(got, _oracle(t, t.wl, scale=1.0), TOL["bf16"], t.wl.name)


def test_a_wait_that_nothing_ends_gives_up_and_reports_it(binding):
    """The bounded wait of the scan kernels, on a barrier nobody arrives on: it must run out after its limit, leave
    DARKATTN_ERR_TIMEOUT in the status word, and the kernel must end normally (the next call works)."""
    status, seconds = binding.darkattn_selftest_wait_limit()
    assert status == binding.ERR_TIMEOUT
    assert 1.5 < seconds < 6.0, seconds
    wl = inputs.small(name="after_timeout", wid=5, B=1, H=1, N=128, d=64, m=128, causal=True, dtype="bf16", backward=False)
    t = inputs.generate(wl)
    _compare(run_gpu(binding, wl, t, path=binding.PATH_TENSOR), _oracle(t, wl), TOL["bf16"], "after_timeout")


def test_mma_cycle_measurement_is_sane(binding):
    """The instrument behind the scan kernels' tensor-pipe accounting: a 128x128x16 bf16 MMA cannot beat the
    pipe's 8192 flop per clock (64 cycles), and none of the forms the kernels use should cost twice that."""
    for variant in range(5):
        per, fixed = binding.darkattn_measure_mma_cycles(variant, False)
        assert 60.0 < per < 128.0, (variant, per)
        assert 0.0 < fixed < 5000.0, (variant, fixed)
    per256, _ = binding.darkattn_measure_mma_cycles(5, False)
    assert 120.0 < per256 < 256.0, per256
    busy, _ = binding.darkattn_measure_mma_cycles(2, True)
    assert 60.0 < busy < 128.0, busy


def test_kernel_timing_reports_every_kernel_of_a_step(binding):
    import torch
    wl = inputs.small(name="timing", wid=91, B=1, H=2, N=512, d=64, m=256, causal=True, dtype="bf16", backward=True)
    t = inputs.generate(wl)
    from tests.util import to_dev
    Q, K, V, M, W, dO = (to_dev(x, torch.bfloat16) for x in (t.Q, t.K, t.V, t.M, t.W, t.dO))
    plan = binding.darkattn_plan(1, 2, 512, 64, 256, causal=True)
    ws = plan.alloc_workspace()
    saved = torch.empty(plan.saved_bytes, dtype=torch.uint8, device="cuda")
    O, dQ, dK, dV = torch.empty_like(V), torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
    dM = torch.empty(M.shape, dtype=torch.float32, device="cuda")
    binding.darkattn_kernel_timing(plan, True)
    for _ in range(2):
        binding.darkattn_forward(plan, Q, K, V, M, W, O, ws, saved=saved)
        binding.darkattn_backward(plan, Q, K, V, M, W, O, dO, dQ, dK, dV, dM, ws, saved=saved)
        times = binding.darkattn_kernel_times(plan)
    expected = 2 * (plan.launches(False) + plan.launches(True))      # as launched while timing is on (one stream)
    binding.darkattn_kernel_timing(plan, False)
    assert plan.launches(True) == expected // 2 - plan.launches(False) + 1     # off: the dM product runs beside, plus a small add kernel
    assert binding.darkattn_last_device_status(plan, ws) == binding.OK
    for name in ("tc_fwd_causal_kernel", "combine_kernel", "tc_bwd_q_kernel", "tc_bwd_k_kernel", "tc_bwd_finish_k_kernel"):
        ms, launches = times[name]
        assert launches == 2 and 0.0 < ms < 1e3, (name, ms, launches)
    assert sum(c for _, c in times.values()) == expected
    plan.destroy()


def test_tensor_path_rejects_uncovered_shapes(binding):
    for kw in (dict(N=200), dict(d=48), dict(m=96)):
        a = dict(B=1, H=1, N=256, d=64, m=128)
        a.update(kw)
        with pytest.raises(binding.DarkAttnError) as e:
            binding.darkattn_plan(a["B"], a["H"], a["N"], a["d"], a["m"], dtype=binding.BF16, path=binding.PATH_TENSOR)
        assert e.value.status == binding.ERR_UNSUPPORTED
        p = binding.darkattn_plan(a["B"], a["H"], a["N"], a["d"], a["m"], dtype=binding.BF16)   # AUTO falls back
        assert p.path == binding.PATH_SIMT
        p.destroy()
