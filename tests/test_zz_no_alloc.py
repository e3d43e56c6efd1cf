"""The forward entry point for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option (a serving loop whose
device memory was fixed at start-up, a plug-in under a framework that owns the device heap).
monarch_fwd_noalloc serves them from an array built into the library.  This file checks,
through the C ABI, that it gives the same result as monarch_fwd - and as the CPU oracle - on
two calls in a row (the second call reuses the array the first one left dirty) and that it
refuses what does not fit.
It is named to be collected last, so a failure here cannot hide another test's result.
"""
import numpy as np
import pytest

import __graft_entry__ as entry
from oracle import monarch_oracle as O
from tests.helpers import assert_close, to_device, to_host64
from paper_2204_00595_b200.inputs import round_to_storage

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import torch
    assert torch.cuda.is_available()
    entry.build()
    import paper_2204_00595_b200 as pkg
    pkg.lib()
    return pkg


def _inputs(m, T, dtype, seed):
    rng = np.random.default_rng(seed)
    n = m * m
    draw = lambda shape, std: round_to_storage(
        rng.standard_normal(shape, dtype=np.float32) * np.float32(std), dtype)
    return draw((T, n), 1.0), draw((m, m, m), m ** -0.5), draw((m, m, m), m ** -0.5)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_noalloc_matches_fwd_on_two_calls_in_a_row(P, dtype):
    import torch
    prev = P.monarch_set_impl(P.IMPL_STAGED)
    try:
        # second case is smaller than the first and of another block size, so it runs on
        # scratch that still holds the first call's intermediate
        for m, T, seed in ((64, 300, 1), (32, 77, 2)):
            n = m * m
            host = _inputs(m, T, dtype, seed)
            x, L, R = (to_device(a, dtype) for a in host)
            code = P.F32 if dtype == "f32" else P.BF16
            ws = P.Workspace(P.monarch_workspace_bytes(P.OP_FWD, T, n, m, code))
            y_ref = torch.full_like(x, float("nan"))
            y_new = torch.full_like(x, float("nan"))
            P.monarch_fwd(x, L, R, y_ref, T, n, m, ws)
            P.monarch_fwd_noalloc(x, L, R, y_new, T, n, m)
            torch.cuda.synchronize()
            assert bool(torch.isfinite(y_new.float()).all())
            assert_close(to_host64(y_new), to_host64(y_ref), dtype, f"noalloc m={m}")
            assert_close(to_host64(y_new), O.fwd(*host), dtype, f"noalloc m={m} against the oracle")
    finally:
        P.monarch_set_impl(prev)


def test_noalloc_rejects_what_does_not_fit(P):
    import torch
    m, n = 64, 4096
    T = P.binding.NOALLOC_SCRATCH_BYTES // (n * 2) + 1
    x = torch.zeros(T, n, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(m, m, m, dtype=torch.bfloat16, device="cuda")
    y = torch.full_like(x, 7.0)
    with pytest.raises(P.MonarchError) as e:
        P.monarch_fwd_noalloc(x, W, W.clone(), y, T, n, m)
    assert e.value.status == 3
    torch.cuda.synchronize()
    assert float(y.float().min()) == 7.0          # nothing was enqueued
    P.monarch_fwd_noalloc(x, W, W.clone(), y, T - 1, n, m)   # the largest size that fits
    torch.cuda.synchronize()
    assert float(y[: T - 1].float().abs().max()) == 0.0
