"""CPU-side checks of the CUDA library: it builds, loads, exports the declared C ABI, and its own
table generator agrees with the oracle (which shares no code with it)."""
import os
import re

import numpy as np
import pytest


@pytest.fixture(scope="module")
def lib():
    from paper_2603_11021_b200 import build
    build.build()
    import paper_2603_11021_b200 as P
    P.load_library()
    return P


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "llvq.h")).read()
    declared = sorted(set(re.findall(r"\b(llvq_[a-z_0-9]+)\s*\(", header)))
    assert declared, "no declarations found"
    L = lib.load_library()
    for name in declared:
        assert hasattr(L, name), name
    assert set(lib.EXPORTS) <= set(declared)


@pytest.mark.parametrize("code", [(2, 2), (3, 3), (2, 13), (2, 53)])
def test_table_generator_agrees_with_oracle(lib, oracle_mod, code):
    ctx = lib.Context(*code, device=-1)                 # host-only context: no GPU needed
    o = oracle_mod.Code(*code)
    assert (ctx.index_bits, ctx.num_points, ctx.num_classes) == (o.W, o.N, o.num_classes)
    step = 1 if o.num_classes < 1000 else 97
    for j in list(range(0, o.num_classes, step)) + [o.num_classes - 1]:
        assert ctx.class_info(j) == o.class_info(j), j
    assert np.array_equal(ctx.golay_table(), oracle_mod.golay_table())
    for n in (0, 1, 3, 8192, 699051):
        want = ((n * o.W + 7) // 8 + 15) // 16 * 16
        assert ctx.index_bytes(n) == want


def test_host_only_context_refuses_to_launch(lib):
    ctx = lib.Context(2, 2, device=-1)
    L = ctx._lib
    assert L.llvq_decode_blocks(ctx._h, 16, 1, 16, None) == 1
    assert L.llvq_last_error(ctx._h, None, None, None) == 1


def test_unsupported_codes_are_rejected(lib):
    import ctypes
    L = lib.load_library()
    h = ctypes.c_void_p()
    for m_lo, m_hi in [(1, 2), (3, 2), (2, 54), (2, 99)]:
        assert L.llvq_create(ctypes.byref(h), m_lo, m_hi, -1) == 3
        assert not h.value
    assert L.llvq_create(None, 2, 2, -1) == 1
