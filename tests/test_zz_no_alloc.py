"""The allocation-free GEMM entry point against the regular one.

Some callers of this library may only launch work: all device memory already belongs to their own pool,
or they sit in a decode loop that cannot afford the device-wide synchronisation an allocation implies.
For them `llvq_gemm_small_batch_noalloc` keeps its split-K scratch in an array built into the library.
This file checks, through the C ABI, that it returns what `llvq_gemm_small_batch` returns and what the CPU
oracle computes, twice in a row with different activations (the built-in array is shared by all calls, so the
second call runs on whatever the first one left there), and that it refuses sizes the array cannot hold.
The kernels themselves hand every scratch word they touch back as zero, so the clearing the entry point does
before each launch only matters after a call that was cut short; no test provokes that.  The file is named to be
collected last.
"""
import numpy as np
import pytest
import torch

import llvq_inputs as gen
from gpu_util import to_dev_bf16, to_dev_f16, to_dev_u8

pytestmark = pytest.mark.gpu

# the two entry points run the same kernel; only the order of the binary32 split-K additions can differ, which
# moves a bf16 output by at most one rounding step: 2^-7 of its value when it sits just above a power of two (both
# sides are bf16 here, so the step is the full spacing, not the half spacing of a comparison with an exact value)
TOL = 2.0 ** -7
# against the binary64 oracle: binary32 accumulation (1e-3) plus the rounding of the bf16 output
TOL_ORACLE = 1e-3 + 2.0 ** -8


def _rel_err(a, ref):
    ref = ref.astype(np.float64)
    return float(np.max(np.abs(a.astype(np.float64) - ref) / np.maximum(np.abs(ref), 1e-3 * np.abs(ref).max())))


@pytest.mark.parametrize("n_out,k_in,batch", [(640, 2048, 16), (300, 1000, 64)])
def test_noalloc_gemm_matches_regular_entry_point_and_oracle_twice(n_out, k_in, batch, code_2_13):
    import paper_2603_11021_b200 as P
    assert torch.cuda.is_available(), "needs a CUDA device; there is no CPU path"
    ctx = P.Context(2, 13, device=0)
    stream, gain, _ = gen.make_layer(ctx.num_points, ctx.index_bits, n_out, k_in, 1, seed=21)
    d_idx, d_gain = to_dev_u8(stream), to_dev_f16(gain)
    y_new = torch.empty((batch, n_out), dtype=torch.bfloat16, device="cuda")     # allocated by the caller, up front
    for call in range(2):
        X = gen.normal_bf16((batch, k_in), seed=30 + call)                        # different activations per call
        d_x = to_dev_bf16(X)
        want = P.llvq_gemm_small_batch(ctx, d_idx, d_gain, n_out, k_in, d_x).float().cpu().numpy()
        y_new.fill_(float("nan"))
        P.llvq_gemm_small_batch_noalloc(ctx, d_idx, d_gain, n_out, k_in, d_x, y_new)
        torch.cuda.synchronize()
        got = y_new.float().cpu().numpy()
        assert np.isfinite(got).all()
        assert _rel_err(got, want) <= TOL, f"call {call}"
        ref = code_2_13.gemm(stream, gain, n_out, k_in, X, threads=4)
        assert _rel_err(got, ref) <= TOL_ORACLE, f"call {call} against the oracle"
    assert P.llvq_last_error(ctx) == (0, 0)


def test_noalloc_gemm_rejects_sizes_beyond_the_builtin_array():
    import paper_2603_11021_b200 as P
    ctx = P.Context(2, 13, device=0)
    buf = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    g = torch.zeros(8, dtype=torch.float16, device="cuda")
    x = torch.zeros(64 * 24, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    L = ctx._lib
    args = (ctx._h, buf.data_ptr(), g.data_ptr())
    # 16385 rows: more than 128 row tiles; 8192 rows at batch 64: 64 * 8192 floats > 262144
    assert L.llvq_gemm_small_batch_noalloc(*args, 16385, 24, x.data_ptr(), 1, y.data_ptr(), None) == 3
    assert L.llvq_gemm_small_batch_noalloc(*args, 8192, 24, x.data_ptr(), 64, y.data_ptr(), None) == 3
    assert L.llvq_gemm_small_batch_noalloc(*args, 8, 24, None, 1, y.data_ptr(), None) == 1
    torch.cuda.synchronize()
