"""The C-ABI library builds, loads and exports every symbol the header declares; host-side
validation rejects unusable arguments before anything is launched (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2607_12789_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    hdr = open(os.path.join(ROOT, "include", "avq_attn.h")).read()
    declared = re.findall(r"AVQ_API\s+[\w\s\*]+?\b(avq_\w+)\s*\(", hdr)
    assert len(declared) >= 9
    assert sorted(declared) == sorted(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name
    assert lib.avq_version() >= 100


def test_status_strings(lib):
    seen = {lib.avq_status_string(s).decode() for s in range(9)}
    assert len(seen) == 9 and "ok" in seen
    assert lib.avq_status_string(99).decode() == "unknown status"


def _prob(**kw):
    base = dict(B=1, H=1, Nq=256, Nk=256, d=64, M=16, C=4, dtype_code=binding.AVQ_F32, scale=0.125, flags=0)
    base.update(kw)
    return binding.problem(**base)


def test_workspace_bytes_and_layout(lib):
    p = _prob()
    n = binding.workspace_bytes(p, 2, 64)
    # header + 2 index arrays + aggregates, each 256-byte aligned
    need = 256 + 2 * 256 * 4 + 16 * 64 * 4 + 16 * 4 + 16 * 4 * 64 * 4 + 16 * 4 * 4
    assert need <= n <= need + 6 * 256
    offs = [ctypes.c_size_t() for _ in range(6)]
    assert lib.avq_workspace_layout(ctypes.byref(p), 2, 64, *[ctypes.byref(o) for o in offs]) == 0
    vals = [o.value for o in offs]
    assert len(set(vals)) == 6 and min(vals) == 256 and all(v % 256 == 0 for v in vals) and max(vals) < n
    pb = _prob(dtype_code=binding.AVQ_BF16, Nq=1024, Nk=1024, M=64)
    assert binding.workspace_bytes(pb, 8, 128) > binding.workspace_bytes(_prob(Nq=1024, Nk=1024, M=64), 8, 128)


@pytest.mark.parametrize("kw,P,bq,want", [
    (dict(B=0), 2, 64, 2), (dict(d=-4), 2, 64, 2), (dict(dtype_code=7), 2, 64, 2), (dict(flags=64), 2, 64, 2),
    (dict(), 17, 64, 2), (dict(), -1, 64, 2), (dict(), 2, 0, 2), (dict(scale=float("nan")), 2, 64, 2),
    (dict(d=6), 2, 64, 3), (dict(d=512), 2, 64, 3), (dict(M=2048), 2, 64, 3), (dict(C=32), 2, 64, 3),
    (dict(), 2, 512, 3), (dict(B=70000), 2, 64, 3),
    (dict(d=256), 2, 256, 3),                                   # CUDA-core attention tile beyond 200 KiB of shared memory
    (dict(dtype_code=binding.AVQ_BF16, d=96), 2, 128, 3), (dict(dtype_code=binding.AVQ_BF16, M=24), 2, 128, 3),
    (dict(dtype_code=binding.AVQ_BF16, C=3), 2, 128, 3), (dict(dtype_code=binding.AVQ_BF16), 2, 64, 3),
])
def test_invalid_problems_are_rejected_on_the_host(lib, kw, P, bq, want):
    p = _prob(**kw)
    assert binding.workspace_bytes(p, P, bq) == 0
    assert lib.avq_workspace_layout(ctypes.byref(p), P, bq, None, None, None, None, None, None) == want
    fake = ctypes.c_void_p(0x1000)
    st = lib.avq_forward(ctypes.byref(p), fake, fake, fake, fake, fake, P, bq, fake, None, None, fake, 1 << 30, None)
    assert st == want


def test_null_misaligned_and_small_workspace_are_rejected_on_the_host(lib):
    p = _prob()
    ok, odd = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1004)
    f = lambda *a: lib.avq_forward(ctypes.byref(p), *a)
    assert f(None, ok, ok, ok, ok, 2, 64, ok, None, None, ok, 1 << 30, None) == 1
    assert f(ok, ok, ok, ok, ok, 2, 64, None, None, None, ok, 1 << 30, None) == 1
    assert f(ok, odd, ok, ok, ok, 2, 64, ok, None, None, ok, 1 << 30, None) == 4
    assert f(ok, ok, ok, ok, ok, 2, 64, ok, None, None, None, 1 << 30, None) == 5
    assert f(ok, ok, ok, ok, ok, 2, 64, ok, None, None, ok, 1000, None) == 5
    assert f(ok, ok, ok, ok, ok, 2, 64, ok, None, None, ctypes.c_void_p(0x1010), 1 << 30, None) == 4
    assert lib.avq_forward(None, ok, ok, ok, ok, ok, 2, 64, ok, None, None, ok, 1 << 30, None) == 1
    assert lib.avq_assign(ctypes.byref(p), ok, ok, None, ok, ok, None) == 1
    assert lib.avq_assign(ctypes.byref(p), ok, ok, ok, odd, ok, None) == 4
    assert lib.avq_aggregate(ctypes.byref(p), ok, ok, ok, ok, ok, ok, None, None) == 1
    assert lib.avq_check(None, None) == 1
    assert lib.avq_forward_host(ctypes.byref(p), None, ok, ok, ok, ok, 2, 64, ok, ok, ok, ok, ok, ok, 1 << 30, None) == 1


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()
