"""The C-ABI library loads, exports every symbol the header declares, and validates descriptors on
the host (no GPU needed: planning touches no device state)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2603_04127_b200 import build
    build.build()
    from paper_2603_04127_b200 import binding as b
    return b


def _declared_symbols(header="darkattn.h"):
    text = open(os.path.join(ROOT, "include", header)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(darkattn_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(binding):
    names = _declared_symbols()
    assert len(names) >= 12
    for n in names:
        assert hasattr(binding.lib, n), n
    assert sorted(binding.EXPORTS) == [n for n in names if n in binding.EXPORTS]
    assert set(names) == set(binding.EXPORTS)
    # the instruments of the benchmark: their own header, their own library
    bench = [n for n in _declared_symbols("darkattn_bench.h")]
    assert set(bench) == set(binding.BENCH_EXPORTS)
    for n in bench:
        assert hasattr(binding.benchlib(), n) and not hasattr(binding.lib, n), n


def test_plan_defaults_and_sizes(binding):
    p = binding.darkattn_plan(1, 1, 256, 64, 64, dtype=binding.F32)
    assert p.path == binding.PATH_SIMT
    assert p.workspace_bytes > 0 and p.workspace_bytes % 256 == 0
    assert p.launches() > 0 and p.launches(True) > p.launches()
    big = binding.darkattn_plan(4, 16, 8192, 128, 256, dtype=binding.BF16, causal=True, path=binding.PATH_SIMT)
    assert big.workspace_bytes < 60e9
    p.destroy(); big.destroy()


@pytest.mark.parametrize("kw", [dict(B=0), dict(N=0), dict(m=0), dict(d=-1), dict(dtype=7), dict(path=9),
                                dict(scale=-1.0), dict(chunk=-4)])
def test_plan_rejects_bad_descriptors(binding, kw):
    args = dict(B=1, H=1, N=128, d=64, m=64, dtype=binding.F32)
    args.update(kw)
    B, H, N, d, m = (args.pop(k) for k in ("B", "H", "N", "d", "m"))
    with pytest.raises(binding.DarkAttnError) as e:
        binding.darkattn_plan(B, H, N, d, m, **args)
    assert e.value.status == binding.ERR_INVALID_ARG


def test_tensor_path_refuses_f32(binding):
    with pytest.raises(binding.DarkAttnError) as e:
        binding.darkattn_plan(1, 1, 256, 64, 256, dtype=binding.F32, path=binding.PATH_TENSOR)
    assert e.value.status == binding.ERR_UNSUPPORTED


def test_null_and_misaligned_pointers_are_rejected_before_launch(binding):
    p = binding.darkattn_plan(1, 1, 128, 64, 64, dtype=binding.F32)
    vp = ctypes.c_void_p
    rc = binding.lib.darkattn_forward(p.handle, None, None, None, None, None, None, None, None, None)
    assert rc == binding.ERR_INVALID_ARG
    a = vp(4096)
    rc = binding.lib.darkattn_forward(p.handle, a, a, a, a, a, a, None, None, None)
    assert rc == binding.ERR_WORKSPACE
    rc = binding.lib.darkattn_forward(p.handle, vp(4100), a, a, a, a, a, None, a, None)
    assert rc == binding.ERR_INVALID_ARG
    assert binding.lib.darkattn_status_string(rc).decode() == "invalid argument"
    p.destroy()
