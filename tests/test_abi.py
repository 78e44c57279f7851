"""CPU-side checks of the C-ABI library: it loads, exports every symbol include/reflex.h declares,
sizes follow the documented layout, and host-side validation rejects bad arguments before anything
is launched (none of these calls reaches a kernel)."""
import ctypes
import os
import re

import pytest

from paper_2607_14695_b200 import binding as rb
from paper_2607_14695_b200 import build as rbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    rbuild.build()
    return rb.load()


def test_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "reflex.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(reflex_[a-z_0-9]+)\s*\(", header))
    assert {"reflex_cache_init_static", "reflex_cache_append_sliding", "reflex_adarmsnorm",
            "reflex_partitioned_attention", "reflex_flow_step"} <= declared
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in reflex.h but not exported"
    assert declared == set(rb.EXPORTS)


def test_sizes(lib):
    d = rb.CacheDesc(18, 64, 8, 1, 256, 816, 32, 50, rb.DTYPE_BF16)
    assert rb.reflex_cache_slab_bytes(d) == 18 * 64 * (816 + 32) * 1 * 256 * 2
    assert rb.reflex_workspace_bytes(d) > 64 * 16
    d32 = rb.CacheDesc(1, 1, 2, 1, 64, 64, 16, 8, rb.DTYPE_F32)
    assert rb.reflex_cache_slab_bytes(d32) == (64 + 16) * 64 * 4
    for bad in (rb.CacheDesc(1, 1, 3, 2, 64, 8, 4, 4, 0),      # Hq % Hkv != 0
                rb.CacheDesc(1, 1, 2, 1, 48, 8, 4, 4, 0),      # head_dim not supported
                rb.CacheDesc(1, 1, 2, 1, 64, 8, 0, 4, 0),      # N < 1
                rb.CacheDesc(1, 1, 2, 1, 64, 8, 4, 4, 7)):     # unknown dtype
        assert rb.reflex_cache_slab_bytes(bad) == 0 and rb.reflex_workspace_bytes(bad) == 0


def test_validation_before_launch(lib):
    fake = ctypes.c_void_p(0x1000)        # aligned, never dereferenced: validation fails first
    odd = ctypes.c_void_p(0x1004)
    err = lambda: lib.reflex_last_error_string().decode()
    # flow step
    assert lib.reflex_flow_step(fake, fake, None, 1, 1, 8, 4, 4, rb.DTYPE_F32, None) == rb.ERR_INVALID_ARG and "k=4" in err()
    assert lib.reflex_flow_step(fake, fake, None, 1, 1, 8, -1, 4, rb.DTYPE_F32, None) == rb.ERR_INVALID_ARG
    assert lib.reflex_flow_step(None, fake, None, 1, 1, 8, 0, 4, rb.DTYPE_F32, None) == rb.ERR_INVALID_ARG
    assert lib.reflex_flow_step(odd, fake, None, 1, 1, 8, 0, 4, rb.DTYPE_F32, None) == rb.ERR_ALIGN
    assert lib.reflex_flow_step(fake, fake, None, 0, 1, 8, 0, 4, rb.DTYPE_F32, None) == rb.ERR_SHAPE
    assert lib.reflex_flow_step(fake, fake, None, 1, 1, 8, 0, 4, 9, None) == rb.ERR_INVALID_ARG
    # adarmsnorm
    a = [fake, fake, fake, fake, fake, fake, fake, None]
    assert lib.reflex_adarmsnorm(*a, 1, 1, 100, 8, 8, 1e-6, 0, None) == rb.ERR_SHAPE          # D % 8
    assert lib.reflex_adarmsnorm(*a, 1, 1, 128, 12, 8, 1e-6, 0, None) == rb.ERR_SHAPE         # Cd % 8
    assert lib.reflex_adarmsnorm(fake, fake, None, None, None, None, None, None, 1, 1, 128, 8, 8, 1e-6, 0, None) == rb.ERR_INVALID_ARG
    assert lib.reflex_adarmsnorm(odd, fake, fake, fake, fake, fake, fake, None, 1, 1, 128, 8, 8, 1e-6, 0, None) == rb.ERR_ALIGN
    assert lib.reflex_adarmsnorm(*a, 1, 1, 128, 8, 8, -1.0, 0, None) == rb.ERR_INVALID_ARG
    # plain projection with residual
    fake2 = ctypes.c_void_p(0x2000)
    assert lib.reflex_linear_residual(None, fake, fake, fake2, fake2, 4, 64, 16, rb.DTYPE_BF16, 3, None) == rb.ERR_INVALID_ARG and "impl" in err()
    assert lib.reflex_linear_residual(None, fake, fake, None, None, 4, 64, 16, rb.DTYPE_BF16, 0, None) == rb.ERR_INVALID_ARG      # out NULL
    assert lib.reflex_linear_residual(None, fake, fake, None, fake, 4, 64, 16, rb.DTYPE_BF16, 0, None) == rb.ERR_INVALID_ARG      # out aliases a
    assert lib.reflex_linear_residual(None, fake, fake, fake2, fake2, 4, 60, 16, rb.DTYPE_BF16, 0, None) == rb.ERR_SHAPE          # K % 8
    assert lib.reflex_linear_residual(None, fake, fake, fake2, fake2, 4, 64, 12, rb.DTYPE_BF16, 0, None) == rb.ERR_SHAPE          # N % 8
    assert lib.reflex_linear_residual(None, fake, fake, fake2, fake2, 0, 64, 16, rb.DTYPE_BF16, 0, None) == rb.ERR_SHAPE          # M < 1
    assert lib.reflex_linear_residual(None, fake, odd, fake2, fake2, 4, 64, 16, rb.DTYPE_BF16, 0, None) == rb.ERR_ALIGN
    assert lib.reflex_linear_residual(None, fake, fake, fake2, fake2, 4, 64, 16, 5, 0, None) == rb.ERR_INVALID_ARG               # dtype
    # gate MLP for all layers
    assert lib.reflex_adarmsnorm_gate(fake, fake, fake, fake, fake, fake, 0, 1, 128, 8, 8, 0, None) == rb.ERR_SHAPE              # L < 1
    assert lib.reflex_adarmsnorm_gate(fake, fake, fake, fake, fake, fake, 1, 1, 128, 8, 1032, 0, None) == rb.ERR_SHAPE           # Hd > 1024
    assert lib.reflex_adarmsnorm_gate(fake, fake, fake, fake, fake, None, 1, 1, 128, 8, 8, 0, None) == rb.ERR_INVALID_ARG
    # cache calls with a NULL handle
    assert lib.reflex_partitioned_attention(None, 0, fake, fake, fake, fake, 1, 0.0, 0, None) == rb.ERR_INVALID_ARG
    assert lib.reflex_cache_init_static(None, None, 0, fake, fake, 0, None, None) == rb.ERR_INVALID_ARG
    assert lib.reflex_cache_append_sliding(None, None, 0, fake, fake, 1, None, None) == rb.ERR_INVALID_ARG
    out = ctypes.c_void_p()
    bad = rb.CacheDesc(1, 1, 3, 2, 64, 8, 4, 4, 0)
    assert lib.reflex_cache_create(ctypes.byref(bad), fake, fake, fake, None, None, ctypes.byref(out)) == rb.ERR_SHAPE
    good = rb.CacheDesc(1, 1, 2, 1, 64, 8, 4, 4, 0)
    assert lib.reflex_cache_create(ctypes.byref(good), None, fake, fake, None, None, ctypes.byref(out)) == rb.ERR_INVALID_ARG
    assert lib.reflex_cache_create(ctypes.byref(good), odd, fake, fake, None, None, ctypes.byref(out)) == rb.ERR_ALIGN
    head0 = (ctypes.c_int32 * 1)(4)
    assert lib.reflex_cache_create(ctypes.byref(good), fake, fake, fake, head0, None, ctypes.byref(out)) == rb.ERR_INVALID_ARG


def test_product_does_not_import_oracle():
    """The package and the bench's product path never reference the oracle."""
    pkg = os.path.join(ROOT, "paper_2607_14695_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "reflex_oracle" not in text and "from oracle" not in text and "import oracle" not in text, fn
