"""Host-buffer entry points against the CPU oracle: same arithmetic as the device calls, with the
library doing the chunked upload / compute / download (needs a B200)."""
import numpy as np
import pytest

import __graft_entry__ as entry
from oracle import monarch_oracle as O
from paper_2204_00595_b200.inputs import round_to_storage
from tests.helpers import assert_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import torch
    assert torch.cuda.is_available()
    entry.build()
    import paper_2204_00595_b200 as pkg
    pkg.lib()
    return pkg


def _host(a, dtype, pin):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    t = t.to(torch.bfloat16) if dtype == "bf16" else t
    return t.pin_memory() if pin else t


# chunk 64 with T = 300 gives five chunks (more than the three staging buffers) and a ragged tail
@pytest.mark.parametrize("m,T,chunk,dtype,pin", [
    (16, 300, 64, "f32", True), (64, 300, 64, "bf16", True), (64, 130, 0, "bf16", False),
    (32, 200, 128, "bf16", True), (64, 0, 64, "bf16", True),
])
def test_host_fwd_bwd(P, m, T, chunk, dtype, pin):
    import torch
    n = m * m
    rng = np.random.default_rng(77 * m + T)

    def draw(shape, std):
        return round_to_storage(rng.standard_normal(shape, dtype=np.float32) * np.float32(std), dtype)

    d = {"x": draw((T, n), 1.0), "dy": draw((T, n), 1.0),
         "L": draw((m, m, m), m ** -0.5), "R": draw((m, m, m), m ** -0.5)}
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    hx, hdy, hL, hR = (_host(d[k], dtype, pin) for k in ("x", "dy", "L", "R"))
    hy = torch.full((T, n), float("nan"), dtype=tdt)
    hdx = torch.full((T, n), float("nan"), dtype=tdt)
    hdL = torch.full((m, m, m), float("nan"), dtype=torch.float32)
    hdR = torch.full((m, m, m), float("nan"), dtype=torch.float32)
    ctx = P.HostContext(max(T, 1), n, m, P.F32 if dtype == "f32" else P.BF16, chunk)
    try:
        ctx.fwd_bwd(hx, hdy, hL, hR, hy, hdx, hdL, hdR, T)
        hy2 = torch.full((T, n), float("nan"), dtype=tdt)
        ctx.fwd(hx, hL, hR, hy2, T)
    finally:
        ctx.close()
    ref_y = O.fwd(d["x"], d["L"], d["R"])
    ref = O.bwd(d["x"], d["dy"], d["L"], d["R"])
    f64 = lambda t: t.to(torch.float32).numpy().astype(np.float64)
    assert_close(f64(hy), ref_y, dtype, "y")
    assert_close(f64(hy2), ref_y, dtype, "y (fwd only)")
    assert_close(f64(hdx), ref["dx"], dtype, "dx")
    assert_close(f64(hdL), ref["dL"], dtype, "dL")
    assert_close(f64(hdR), ref["dR"], dtype, "dR")


def test_host_rejects_bad_arguments(P):
    import torch
    with pytest.raises(P.MonarchError):
        P.HostContext(128, 4096, 64, P.BF16, 100)          # chunk not a multiple of 64
    with pytest.raises(P.MonarchError):
        P.HostContext(128, 4096, 48, P.BF16, 64)           # unsupported m
    ctx = P.HostContext(64, 256, 16, P.F32, 64)
    x = torch.zeros(128, 256)
    w = torch.zeros(16, 16, 16)
    with pytest.raises(P.MonarchError):
        ctx.fwd(x, w, w, torch.empty_like(x), 128)         # more tokens than the context was made for
    ctx.close()
