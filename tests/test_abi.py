"""The C ABI: the library builds, loads without a GPU, and exports every function the header declares."""
import ctypes as C
import os
import re

import pytest

from paper_2402_13720_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def header_functions():
    text = open(os.path.join(ROOT, "include", "ouro.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ouro_[a-z_]+)\s*\(", text)) - {"ouro_drafter_fn"})


def test_every_declared_function_is_exported_and_bound(lib):
    names = header_functions()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} declared in ouro.h but not exported"
    assert set(names) == set(binding.exported_names())


def test_status_texts(lib):
    assert lib.ouro_strerror(0) == b"ok"
    assert all(lib.ouro_strerror(s) for s in range(8))


def test_workspace_bytes_and_argument_checks(lib):
    for name in ("C1", "C2", "C3", "C4", "C5"):
        t, d, p, _ = synth.config(name)
        td, pd = binding.desc_c(t), binding.params_c(p)
        dd = binding.desc_c(d) if d is not None else None
        n = lib.ouro_workspace_bytes(C.byref(td), C.byref(dd) if dd else None, C.byref(pd))
        assert 0 < n < 2 << 30, (name, n)
    bad = binding.desc_c(t)
    bad.head_dim = 48
    assert lib.ouro_workspace_bytes(C.byref(bad), None, C.byref(pd)) == 0
    pbad = binding.params_c(p)
    pbad.K = 16; pbad.beta = 16          # 1 + gamma + 16*15 rows > OURO_MAX_ROWS
    assert lib.ouro_workspace_bytes(C.byref(td), None, C.byref(pbad)) == 0
    pbad = binding.params_c(p)
    pbad.pool_sets = 48                   # not a power of two
    assert lib.ouro_workspace_bytes(C.byref(td), None, C.byref(pbad)) == 0


def test_create_rejects_bad_arguments_without_a_gpu(lib):
    t, d, p, _ = synth.config("C1")
    td, pd = binding.desc_c(t), binding.params_c(p)
    ctx = C.c_void_p()
    mem = binding.ModelMemC()
    rc = lib.ouro_create(C.byref(td), C.byref(mem), None, None, C.byref(pd), 256, 1 << 20, None, C.byref(ctx))
    assert rc == binding.OURO_EINVAL and not ctx.value
    assert b"target" in lib.ouro_last_error(None)
    assert lib.ouro_destroy(None) == binding.OURO_EINVAL
    assert lib.ouro_verify_forward(None, 0, None, None) == binding.OURO_EINVAL


def test_engine_needs_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    t, d, p, _ = synth.config("C1")
    with pytest.raises(RuntimeError):
        binding.Engine(t, {}, p)
