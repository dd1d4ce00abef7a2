"""CPU-side checks of the C ABI: the library builds, loads, exports every declared symbol,
and validates its arguments before touching a device."""
import ctypes
import os
import re

import pytest

import paper_2605_13473_b200 as osdn
from paper_2605_13473_b200 import binding
from paper_2605_13473_b200.build import build
from paper_2605_13473_b200.synth import OsdnHyper

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build()
    return osdn.load_library()


def test_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "osdn.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(osdn_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS), declared ^ set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_workspace_sizes_and_validation(lib):
    hy = OsdnHyper()
    p = osdn.make_params(B=8, T=2048, H=8, K=128, V=128, io_dtype="bf16", hyper=hy)
    fwd_bytes = osdn.osdn_workspace_bytes(p, False)
    bwd_bytes = osdn.osdn_workspace_bytes(p, True)
    assert 0 < fwd_bytes < bwd_bytes < 8 << 30
    assert osdn.osdn_host_staging_bytes(p, True) > bwd_bytes
    for bad in (dict(K=96), dict(V=32), dict(T=0)):
        kw = dict(B=1, T=64, H=1, K=64, V=64)
        kw.update(bad)
        q = osdn.make_params(io_dtype="fp32", hyper=hy, **kw)
        assert osdn.osdn_workspace_bytes(q, False) == 0
    q = osdn.make_params(B=1, T=64, H=1, K=64, V=64, io_dtype="fp32", hyper=hy)
    q.chunk = 32
    assert osdn.osdn_workspace_bytes(q, False) == 0


def test_calls_reject_bad_arguments_before_any_launch(lib):
    hy = OsdnHyper()
    p = osdn.make_params(B=1, T=64, H=1, K=64, V=64, io_dtype="fp32", hyper=hy)
    null = ctypes.c_void_p(None)
    rc = lib.osdn_fwd(ctypes.byref(p), *([null] * 11), null, ctypes.c_size_t(0), null)
    assert rc == -1 and osdn.status_string(rc) == "invalid argument"
    fake = ctypes.c_void_p(0x1000)      # never dereferenced: validation fails first
    odd = ctypes.c_void_p(0x1004)
    rc = lib.osdn_fwd(ctypes.byref(p), odd, fake, fake, fake, fake, null, null, null, fake, null, null,
                      fake, ctypes.c_size_t(1 << 30), null)
    assert rc == -3
    rc = lib.osdn_fwd(ctypes.byref(p), fake, fake, fake, fake, fake, null, null, null, fake, null, null,
                      fake, ctypes.c_size_t(16), null)
    assert rc == -4
    p.apf_mode = 2
    rc = lib.osdn_fwd(ctypes.byref(p), fake, fake, fake, fake, fake, null, null, null, fake, null, null,
                      fake, ctypes.c_size_t(1 << 30), null)
    assert rc == -1                     # separate retention requested but not given
    p.apf_mode = 3
    rc = lib.osdn_fwd(ctypes.byref(p), fake, fake, fake, fake, fake, null, null, null, fake, null, null,
                      fake, ctypes.c_size_t(1 << 30), null)
    assert rc == -1                     # vector retention requested but not given
    p.apf_mode = 4
    assert osdn.osdn_workspace_bytes(p, False) == 0   # no such retention mode
    p.apf_mode = 1
    p.nseq = 3                          # var-len without cu_seqlens
    rc = lib.osdn_precond_update(ctypes.byref(p), fake, fake, fake, null, null, fake, null)
    assert rc == -1
    assert osdn.status_string(-2) == "unsupported shape"
    # the residual-ratio diagnostic: no output requested, misaligned output
    pr = osdn.make_params(B=1, T=64, H=1, K=64, V=64, io_dtype="fp32", hyper=hy)
    rc = lib.osdn_residual_ratio(ctypes.byref(pr), fake, fake, fake, null, null, null, null, null)
    assert rc == -1
    rc = lib.osdn_residual_ratio(ctypes.byref(pr), fake, fake, fake, null, odd, null, null, null)
    assert rc == -3
    # the recurrent step: missing cache, misaligned pointer, missing separate retention, packed batch
    p = osdn.make_params(B=2, T=1, H=1, K=128, V=128, io_dtype="bf16", hyper=hy)
    rc = lib.osdn_decode_step(ctypes.byref(p), fake, fake, fake, fake, fake, null, null, fake, fake, null)
    assert rc == -1
    rc = lib.osdn_decode_step(ctypes.byref(p), fake, fake, fake, fake, fake, null, odd, fake, fake, null)
    assert rc == -3
    p.apf_mode = 2
    rc = lib.osdn_decode_step(ctypes.byref(p), fake, fake, fake, fake, fake, null, fake, fake, fake, null)
    assert rc == -1
    p.apf_mode = 1
    p.K = 96
    rc = lib.osdn_decode_step(ctypes.byref(p), fake, fake, fake, fake, fake, null, fake, fake, fake, null)
    assert rc == -2


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(RuntimeError, match="no fallback"):
        osdn.load_library(str(tmp_path / "libosdn.so"))
