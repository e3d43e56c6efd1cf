"""Parity of the CUDA library against the CPU oracle, through the C ABI (needs a B200)."""
import numpy as np
import pytest

import __graft_entry__ as entry
from oracle import monarch_oracle as O
from paper_2204_00595_b200.inputs import CONFIGS, make_inputs, round_to_storage
from tests.helpers import assert_close, rel_errors, to_device, to_host64

pytestmark = pytest.mark.gpu

GUARD = 64  # sentinel elements after every output


@pytest.fixture(scope="module")
def P():
    import torch
    assert torch.cuda.is_available()
    entry.build()
    import paper_2204_00595_b200 as pkg
    pkg.lib()
    return pkg


@pytest.fixture(params=["staged", "auto"])
def impl(request, P):
    prev = P.monarch_set_impl(P.IMPL_STAGED if request.param == "staged" else P.IMPL_AUTO)
    yield request.param
    P.monarch_set_impl(prev)


def _skip_if_same_family(P, impl, op, m, code):
    if impl == "auto" and P.monarch_impl_name(op, m, code) == "staged-simt":
        pytest.skip("auto selects the staged family here (already covered)")


def _guarded(shape, dtype):
    """Output buffer filled with NaN plus a sentinel tail that must stay untouched."""
    import torch
    numel = int(np.prod(shape))
    flat = torch.full((numel + GUARD,), float("nan"), dtype=dtype, device="cuda")
    flat[numel:] = 1024.0
    return flat, flat[:numel].view(*shape)


def _check_guard(flat, what):
    tail = flat[-GUARD:].float().cpu().numpy()
    assert np.all(tail == 1024.0), f"{what}: wrote past the end of the output"


def _code(P, dtype):
    return P.F32 if dtype == "f32" else P.BF16


def _tdtype(dtype):
    import torch
    return torch.float32 if dtype == "f32" else torch.bfloat16


def _small_inputs(m, T, dtype, seed):
    rng = np.random.default_rng(seed)
    n = m * m
    std_w = 1.0 / np.sqrt(m)

    def draw(shape, std):
        return round_to_storage(rng.standard_normal(shape, dtype=np.float32) * np.float32(std), dtype)

    return {
        "x": draw((T, n), 1.0), "dy": draw((T, n), 1.0),
        "L": draw((m, m, m), std_w), "R": draw((m, m, m), std_w),
        "L2": draw((m, m, m), std_w), "R2": draw((m, m, m), std_w),
        "b1": draw((n,), np.sqrt(0.02)), "b2": draw((n,), np.sqrt(0.02)),
    }


SMALL = [(16, T) for T in (1, 7, 63, 64, 65, 129, 300)] + \
        [(32, T) for T in (1, 65, 129, 257)] + \
        [(64, T) for T in (1, 63, 130, 257)] + \
        [(128, T) for T in (1, 70, 129)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("m,T", SMALL)
def test_fwd_bwd_small(P, impl, m, T, dtype):
    import torch
    code = _code(P, dtype)
    _skip_if_same_family(P, impl, P.OP_FWD, m, code)
    n = m * m
    d = _small_inputs(m, T, dtype, seed=1000 * m + T)
    x, dy, L, R = (to_device(d[k], dtype) for k in ("x", "dy", "L", "R"))
    yf, y = _guarded((T, n), _tdtype(dtype))
    dxf, dx = _guarded((T, n), _tdtype(dtype))
    dLf, dL = _guarded((m, m, m), torch.float32)
    dRf, dR = _guarded((m, m, m), torch.float32)
    ws = P.Workspace(max(P.monarch_workspace_bytes(op, T, n, m, code) for op in range(3)))
    P.monarch_fwd(x, L, R, y, T, n, m, ws)
    P.monarch_bwd_dx(dy, L, R, dx, T, n, m, ws)
    P.monarch_bwd_dw(x, dy, L, R, dL, dR, 0, T, n, m, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    ref_y = O.fwd(d["x"], d["L"], d["R"])
    ref = O.bwd(d["x"], d["dy"], d["L"], d["R"])
    assert_close(to_host64(y), ref_y, dtype, "y")
    assert_close(to_host64(dx), ref["dx"], dtype, "dx")
    assert_close(to_host64(dL), ref["dL"], dtype, "dL")
    assert_close(to_host64(dR), ref["dR"], dtype, "dR")
    for flat, what in ((yf, "y"), (dxf, "dx"), (dLf, "dL"), (dRf, "dR")):
        _check_guard(flat, what)
    # accumulate = 1 adds to the previous contents
    P.monarch_bwd_dw(x, dy, L, R, dL, dR, 1, T, n, m, ws)
    torch.cuda.synchronize()
    assert_close(to_host64(dL), 2 * ref["dL"], dtype, "dL accumulate")
    assert_close(to_host64(dR), 2 * ref["dR"], dtype, "dR accumulate")


@pytest.mark.parametrize("saved", [False, True])
@pytest.mark.parametrize("m,T,dtype", [(16, 65, "f32"), (32, 129, "bf16"), (32, 64 * 150 + 7, "bf16"), (64, 1, "bf16"),
                                       (64, 130, "bf16"), (64, 257, "bf16"), (128, 70, "bf16")])
def test_bwd_one_call(P, impl, m, T, dtype, saved):
    """monarch_bwd = monarch_bwd_dx + monarch_bwd_dw, with or without the forward call's workspace."""
    import torch
    code = _code(P, dtype)
    _skip_if_same_family(P, impl, P.OP_BWD, m, code)
    n = m * m
    d = _small_inputs(m, T, dtype, seed=77 * m + T)
    x, dy, L, R = (to_device(d[k], dtype) for k in ("x", "dy", "L", "R"))
    yf, y = _guarded((T, n), _tdtype(dtype))
    dxf, dx = _guarded((T, n), _tdtype(dtype))
    dLf, dL = _guarded((m, m, m), torch.float32)
    dRf, dR = _guarded((m, m, m), torch.float32)
    ws_f = P.Workspace(P.monarch_workspace_bytes(P.OP_FWD, T, n, m, code))
    ws_b = P.Workspace(P.monarch_workspace_bytes(P.OP_BWD, T, n, m, code))
    P.monarch_fwd(x, L, R, y, T, n, m, ws_f)
    P.monarch_bwd(x, dy, L, R, dx, dL, dR, 0, T, n, m, ws_b, fwd_workspace=ws_f if saved else None)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws_f) == 0 and P.monarch_last_device_status(ws_b) == 0
    ref = O.bwd(d["x"], d["dy"], d["L"], d["R"])
    assert_close(to_host64(y), O.fwd(d["x"], d["L"], d["R"]), dtype, "y")
    assert_close(to_host64(dx), ref["dx"], dtype, "dx")
    assert_close(to_host64(dL), ref["dL"], dtype, "dL")
    assert_close(to_host64(dR), ref["dR"], dtype, "dR")
    for flat, what in ((yf, "y"), (dxf, "dx"), (dLf, "dL"), (dRf, "dR")):
        _check_guard(flat, what)
    P.monarch_bwd(x, dy, L, R, dx, dL, dR, 1, T, n, m, ws_b, fwd_workspace=ws_f if saved else None)
    torch.cuda.synchronize()
    assert_close(to_host64(dL), 2 * ref["dL"], dtype, "dL accumulate")
    assert_close(to_host64(dR), 2 * ref["dR"], dtype, "dR accumulate")


@pytest.mark.parametrize("T", [1, 130, 64 * 40 - 63, 8192])
def test_bwd_m64_fixed_summation_order(P, T):
    """monarch_set_deterministic(1): dL and dR of the fused m = 64 backward are sums in a fixed order - two runs
    from different initial contents give the same bits, both calls (monarch_bwd, monarch_bwd_dw) agree with the
    oracle, accumulate = 1 adds to what is there, and a workspace sized before the switch is refused."""
    import torch
    m, dtype, code = 64, "bf16", P.BF16
    n = m * m
    d = _small_inputs(m, T, dtype, seed=9100 + T)
    x, dy, L, R = (to_device(d[k], dtype) for k in ("x", "dy", "L", "R"))
    ref = O.bwd(d["x"], d["dy"], d["L"], d["R"])
    small = P.monarch_workspace_bytes(P.OP_BWD, T, n, m, code)
    prev = P.monarch_set_deterministic(True)
    try:
        assert P.monarch_impl_name(P.OP_BWD, m, code) == "fused-tcgen05"
        nb = P.monarch_workspace_bytes(P.OP_BWD, T, n, m, code)
        assert nb > small
        ws_f = P.Workspace(P.monarch_workspace_bytes(P.OP_FWD, T, n, m, code))
        ws_b = P.Workspace(nb)
        ws_w = P.Workspace(P.monarch_workspace_bytes(P.OP_BWD_DW, T, n, m, code))
        y = torch.empty_like(x)
        dx = torch.empty_like(x)
        P.monarch_fwd(x, L, R, y, T, n, m, ws_f)
        runs = []
        for fill, saved in ((float("nan"), True), (123.0, False), (-7.0, True)):
            dL = torch.full((m, m, m), fill, device="cuda")
            dR = torch.full((m, m, m), fill, device="cuda")
            P.monarch_bwd(x, dy, L, R, dx, dL, dR, 0, T, n, m, ws_b, fwd_workspace=ws_f if saved else None)
            torch.cuda.synchronize()
            assert P.monarch_last_device_status(ws_b) == 0
            runs.append((dL.clone(), dR.clone()))
        for dL, dR in runs[1:]:
            assert torch.equal(dL, runs[0][0]) and torch.equal(dR, runs[0][1])
        assert_close(to_host64(dx), ref["dx"], dtype, "dx")
        assert_close(to_host64(runs[0][0]), ref["dL"], dtype, "dL fixed order")
        assert_close(to_host64(runs[0][1]), ref["dR"], dtype, "dR fixed order")
        # weight gradients alone: same partial sums, same order
        dL = torch.full((m, m, m), float("nan"), device="cuda")
        dR = torch.full((m, m, m), float("nan"), device="cuda")
        P.monarch_bwd_dw(x, dy, L, R, dL, dR, 0, T, n, m, ws_w)
        P.monarch_bwd_dw(x, dy, L, R, dL, dR, 1, T, n, m, ws_w)
        torch.cuda.synchronize()
        assert P.monarch_last_device_status(ws_w) == 0
        assert_close(to_host64(dL), 2 * ref["dL"], dtype, "dL accumulate, fixed order")
        assert_close(to_host64(dR), 2 * ref["dR"], dtype, "dR accumulate, fixed order")
        with pytest.raises(P.MonarchError):
            P.monarch_bwd(x, dy, L, R, dx, dL, dR, 0, T, n, m, P.Workspace(small))
    finally:
        P.monarch_set_deterministic(prev)
    assert P.monarch_workspace_bytes(P.OP_BWD, T, n, m, code) == small


def test_m32_backward_runs_on_the_tensor_cores(P):
    """bf16 m = 32: dL and dR come from the tcgen05 token-reduction kernel (128-column windows whose diagonal 32 x 32
    sub-blocks are the blocks' sums), not from the CUDA-core kernel - by name and against the oracle, on a token count
    with a ragged last tile."""
    import torch
    m, T, dtype, code = 32, 64 * 9 + 5, "bf16", P.BF16
    n = m * m
    for op in (P.OP_BWD, P.OP_BWD_DW, P.OP_BWD_DX):
        assert P.monarch_impl_name(op, m, code) == "staged-tcgen05"
    d = _small_inputs(m, T, dtype, seed=3232)
    x, dy, L, R = (to_device(d[k], dtype) for k in ("x", "dy", "L", "R"))
    dL = torch.full((m, m, m), float("nan"), device="cuda")
    dR = torch.full((m, m, m), float("nan"), device="cuda")
    ws = P.Workspace(P.monarch_workspace_bytes(P.OP_BWD_DW, T, n, m, code))
    P.monarch_bwd_dw(x, dy, L, R, dL, dR, 0, T, n, m, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    ref = O.bwd(d["x"], d["dy"], d["L"], d["R"])
    assert_close(to_host64(dL), ref["dL"], dtype, "m32 dL")
    assert_close(to_host64(dR), ref["dR"], dtype, "m32 dR")


# Token counts around the persistent kernels' schedule boundaries: 18 teams of 8 CTAs (m = 64: one, two and
# "two and a bit" tiles per team), 148 CTAs (m = 32), each with a ragged last tile.
@pytest.mark.parametrize("m,T", [(64, 64 * 18 - 1), (64, 64 * 18 + 1), (64, 64 * 36 + 5), (64, 64 * 40 - 63),
                                 (32, 64 * 148 - 1), (32, 64 * 148 + 1), (32, 64 * 300 + 3)])
def test_schedule_boundaries(P, m, T):
    import torch
    dtype = "bf16"
    code = P.BF16
    n = m * m
    d = _small_inputs(m, T, dtype, seed=4242 + T)
    x, dy, L, R, L2, R2, b1, b2 = (to_device(d[k], dtype) for k in ("x", "dy", "L", "R", "L2", "R2", "b1", "b2"))
    rows = _sample_tokens(T, 96, 11) if T > 96 else np.arange(T)
    rows = np.unique(np.concatenate([rows, np.arange(T - 70, T)]))          # always include the ragged tail
    yf, y = _guarded((T, n), torch.bfloat16)
    ws = P.Workspace(max(P.monarch_workspace_bytes(P.OP_FWD, T, n, m, code), 256))
    P.monarch_fwd(x, L, R, y, T, n, m, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    yh = to_host64(y)
    assert np.isfinite(yh).all()
    assert_close(yh[rows], O.fwd(d["x"][rows], d["L"], d["R"]), dtype, "y")
    _check_guard(yf, "y")
    if m != 64:
        return
    dxf, dx = _guarded((T, n), torch.bfloat16)
    dL = torch.full((m, m, m), float("nan"), dtype=torch.float32, device="cuda")
    dR = torch.full_like(dL, float("nan"))
    ws_b = P.Workspace(P.monarch_workspace_bytes(P.OP_BWD, T, n, m, code))
    P.monarch_bwd(x, dy, L, R, dx, dL, dR, 0, T, n, m, ws_b, fwd_workspace=ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws_b) == 0
    ref = O.bwd(d["x"], d["dy"], d["L"], d["R"])
    dxh = to_host64(dx)
    assert np.isfinite(dxh).all()
    assert_close(dxh[rows], ref["dx"][rows], dtype, "dx")
    assert_close(to_host64(dL), ref["dL"], dtype, "dL")
    assert_close(to_host64(dR), ref["dR"], dtype, "dR")
    _check_guard(dxf, "dx")
    ws_m = P.Workspace(P.monarch_workspace_bytes(P.OP_MLP_FWD, T, n, m, code))
    P.monarch_mlp_fwd(x, L, R, b1, L2, R2, b2, y, T, n, m, ws_m)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws_m) == 0
    ref_m = O.mlp_fwd(d["x"][rows], d["L"], d["R"], d["b1"], d["L2"], d["R2"], d["b2"])
    assert_close(to_host64(y)[rows], ref_m, dtype, "mlp y")
    _check_guard(yf, "mlp y")


def test_workspace_reuse_across_sizes(P):
    """One workspace, many calls of different sizes: the per-tile dependency counters must be back at zero after
    every call, whatever mix of calls and token counts came before."""
    import torch
    m, n, dtype, code = 64, 4096, "bf16", P.BF16
    Tmax = 1300
    d = _small_inputs(m, Tmax, dtype, seed=99)
    L, R = to_device(d["L"], dtype), to_device(d["R"], dtype)
    ws = P.Workspace(max(P.monarch_workspace_bytes(op, Tmax, n, m, code)
                         for op in (P.OP_FWD, P.OP_BWD_DX, P.OP_BWD_DW, P.OP_BWD, P.OP_MLP_FWD)))
    ws_f = P.Workspace(P.monarch_workspace_bytes(P.OP_FWD, Tmax, n, m, code))
    for T in (257, 64, 1300, 130, 1153, 1):
        x, dy = to_device(d["x"][:T], dtype), to_device(d["dy"][:T], dtype)
        y, dx = torch.empty_like(x), torch.empty_like(x)
        dL = torch.empty(m, m, m, dtype=torch.float32, device="cuda")
        dR = torch.empty_like(dL)
        ref_y = O.fwd(d["x"][:T], d["L"], d["R"])
        ref = O.bwd(d["x"][:T], d["dy"][:T], d["L"], d["R"])
        P.monarch_fwd(x, L, R, y, T, n, m, ws)
        assert_close(to_host64(y), ref_y, dtype, f"y T={T}")
        P.monarch_bwd_dx(dy, L, R, dx, T, n, m, ws)
        assert_close(to_host64(dx), ref["dx"], dtype, f"dx T={T}")
        P.monarch_bwd_dw(x, dy, L, R, dL, dR, 0, T, n, m, ws)
        assert_close(to_host64(dL), ref["dL"], dtype, f"dL T={T}")
        assert_close(to_host64(dR), ref["dR"], dtype, f"dR T={T}")
        P.monarch_fwd(x, L, R, y, T, n, m, ws_f)
        P.monarch_bwd(x, dy, L, R, dx, dL, dR, 0, T, n, m, ws, fwd_workspace=ws_f)
        assert_close(to_host64(dx), ref["dx"], dtype, f"dx one call T={T}")
        assert_close(to_host64(dL), ref["dL"], dtype, f"dL one call T={T}")
        assert_close(to_host64(dR), ref["dR"], dtype, f"dR one call T={T}")
        torch.cuda.synchronize()
        assert P.monarch_last_device_status(ws) == 0 and P.monarch_last_device_status(ws_f) == 0


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("m,T", [(16, 5), (32, 129), (64, 257), (128, 66)])
def test_mlp_small(P, impl, m, T, dtype):
    import torch
    code = _code(P, dtype)
    _skip_if_same_family(P, impl, P.OP_MLP_FWD, m, code)
    n = m * m
    d = _small_inputs(m, T, dtype, seed=77 * m + T)
    t = {k: to_device(d[k], dtype) for k in ("x", "L", "R", "b1", "L2", "R2", "b2")}
    yf, y = _guarded((T, n), _tdtype(dtype))
    ws = P.Workspace(P.monarch_workspace_bytes(P.OP_MLP_FWD, T, n, m, code))
    P.monarch_mlp_fwd(t["x"], t["L"], t["R"], t["b1"], t["L2"], t["R2"], t["b2"], y, T, n, m, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    ref = O.mlp_fwd(d["x"], d["L"], d["R"], d["b1"], d["L2"], d["R2"], d["b2"])
    assert_close(to_host64(y), ref, dtype, "mlp y")
    _check_guard(yf, "mlp y")


MLP_GRADS = ("dL1", "dR1", "db1", "dL2", "dR2", "db2")


def _mlp_bwd_buffers(m, T, dtype):
    import torch
    n = m * m
    bufs = {"dx": _guarded((T, n), _tdtype(dtype))}
    for k in MLP_GRADS:
        bufs[k] = _guarded((n,) if k.startswith("db") else (m, m, m), torch.float32)
    return bufs


def _call_mlp_bwd(P, t, bufs, accumulate, T, n, m, ws):
    P.monarch_mlp_bwd(t["x"], t["dy"], t["L"], t["R"], t["b1"], t["L2"], t["R2"], bufs["dx"][1],
                      *(bufs[k][1] for k in MLP_GRADS), accumulate, T, n, m, ws)


def _assert_mlp_grads(bufs, ref, dtype, what, factor=1.0):
    for k in MLP_GRADS:
        got, want = to_host64(bufs[k][1]), factor * ref[k]
        if k.startswith("db"):                 # one problem instance: the whole bias vector
            got, want = got[None, :], want[None, :]
        assert_close(got, want, dtype, f"{what} {k}")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("m,T", [(16, 5), (32, 129), (64, 64), (64, 257), (128, 66)])
def test_mlp_bwd_small(P, impl, m, T, dtype):
    import torch
    code = _code(P, dtype)
    _skip_if_same_family(P, impl, P.OP_MLP_BWD, m, code)
    n = m * m
    d = _small_inputs(m, T, dtype, seed=91 * m + T)
    t = {k: to_device(d[k], dtype) for k in ("x", "dy", "L", "R", "b1", "L2", "R2")}
    bufs = _mlp_bwd_buffers(m, T, dtype)
    ws = P.Workspace(P.monarch_workspace_bytes(P.OP_MLP_BWD, T, n, m, code))
    _call_mlp_bwd(P, t, bufs, 0, T, n, m, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    ref = O.mlp_bwd(d["x"], d["dy"], d["L"], d["R"], d["b1"], d["L2"], d["R2"])
    assert_close(to_host64(bufs["dx"][1]), ref["dx"], dtype, "mlp dx")
    _assert_mlp_grads(bufs, ref, dtype, "mlp")
    for k, (flat, _) in bufs.items():
        _check_guard(flat, f"mlp {k}")
    # accumulate = 1 adds to the previous contents of the six parameter gradients
    _call_mlp_bwd(P, t, bufs, 1, T, n, m, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    assert_close(to_host64(bufs["dx"][1]), ref["dx"], dtype, "mlp dx (second call)")
    _assert_mlp_grads(bufs, ref, dtype, "mlp accumulate", factor=2.0)


def test_mlp_bwd_zero_tokens(P, impl):
    import torch
    m, n = 64, 4096
    t = {k: torch.zeros(s, dtype=torch.bfloat16, device="cuda")
         for k, s in (("x", (1, n)), ("dy", (1, n)), ("L", (m, m, m)), ("R", (m, m, m)), ("b1", (n,)),
                      ("L2", (m, m, m)), ("R2", (m, m, m)))}
    bufs = _mlp_bwd_buffers(m, 1, "bf16")
    for k in MLP_GRADS:
        bufs[k][1].fill_(5.0)
    ws = P.Workspace(P.monarch_workspace_bytes(P.OP_MLP_BWD, 0, n, m, P.BF16))
    _call_mlp_bwd(P, t, bufs, 1, 0, n, m, ws)
    torch.cuda.synchronize()
    assert all(float(bufs[k][1].min()) == 5.0 for k in MLP_GRADS)
    _call_mlp_bwd(P, t, bufs, 0, 0, n, m, ws)
    torch.cuda.synchronize()
    assert all(float(bufs[k][1].abs().max()) == 0.0 for k in MLP_GRADS)
    assert P.monarch_last_device_status(ws) == 0


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_zero_tokens(P, impl, dtype):
    import torch
    m, n = 32, 1024
    code = _code(P, dtype)
    td = _tdtype(dtype)
    x = torch.zeros(1, n, dtype=td, device="cuda")
    W = torch.zeros(m, m, m, dtype=td, device="cuda")
    y = torch.full((1, n), 3.0, dtype=td, device="cuda")
    dL = torch.full((m, m, m), 5.0, dtype=torch.float32, device="cuda")
    dR = torch.full((m, m, m), 5.0, dtype=torch.float32, device="cuda")
    ws = P.Workspace(1 << 20)
    P.monarch_fwd(x, W, W.clone(), y, 0, n, m, ws)
    P.monarch_bwd_dw(x, x.clone(), W, W.clone(), dL, dR, 1, 0, n, m, ws)
    torch.cuda.synchronize()
    assert float(y.float().min()) == 3.0 and float(dL.min()) == 5.0
    P.monarch_bwd_dw(x, x.clone(), W, W.clone(), dL, dR, 0, 0, n, m, ws)
    torch.cuda.synchronize()
    assert float(dL.abs().max()) == 0.0 and float(dR.abs().max()) == 0.0
    for mm in (32, 64):             # the one-call backward defines dL, dR for an empty batch too
        g = torch.full((2, mm, mm, mm), 5.0, dtype=torch.float32, device="cuda")
        xx = torch.zeros(1, mm * mm, dtype=td, device="cuda")
        Wm = torch.zeros(mm, mm, mm, dtype=td, device="cuda")
        wsb = P.Workspace(max(P.monarch_workspace_bytes(P.OP_BWD, 0, mm * mm, mm, code), 256))
        P.monarch_bwd(xx, xx.clone(), Wm, Wm.clone(), xx.clone(), g[0], g[1], 0, 0, mm * mm, mm, wsb)
        torch.cuda.synchronize()
        assert float(g.abs().max()) == 0.0


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("m", [16, 32])
def test_hadamard_closed_form_exact(P, impl, m, dtype):
    """All blocks H_m (Sylvester): M = H_n, y[a] = sum_b (-1)^popcount(a&b) x[b], exactly."""
    import torch
    code = _code(P, dtype)
    _skip_if_same_family(P, impl, P.OP_FWD, m, code)
    n = m * m
    H = np.array([[1.0]])
    while H.shape[0] < m:
        H = np.block([[H, H], [H, -H]])
    W = np.stack([H] * m).astype(np.float32)
    rng = np.random.default_rng(5)
    T = 70
    x = np.zeros((T, n), dtype=np.float32)
    for t in range(T):                       # a few +-1 entries: every sum is a small integer
        idx = rng.choice(n, size=12, replace=False)
        x[t, idx] = rng.choice([-1.0, 1.0], size=12)
    xd, Wd = to_device(x, dtype), to_device(W, dtype)
    y = torch.empty_like(xd)
    ws = P.Workspace(P.monarch_workspace_bytes(P.OP_FWD, T, n, m, code))
    P.monarch_fwd(xd, Wd, Wd.clone(), y, T, n, m, ws)
    torch.cuda.synchronize()
    a = np.arange(n)
    pc = np.array([[bin(p & q).count("1") & 1 for q in a] for p in a])
    Hn = 1.0 - 2.0 * pc
    assert np.array_equal(to_host64(y), x.astype(np.float64) @ Hn.T)


def test_workspace_too_small_is_reported(P):
    import torch
    m, n, T = 16, 256, 64
    x = torch.zeros(T, n, device="cuda")
    W = torch.zeros(m, m, m, device="cuda")
    y = torch.empty_like(x)
    ws = P.Workspace(256)
    with pytest.raises(P.MonarchError) as e:
        P.monarch_fwd(x, W, W.clone(), y, T, n, m, (ws.ptr, 256))
    assert e.value.status == 3 or P.monarch_workspace_bytes(P.OP_FWD, T, n, m, P.F32) <= 256


# ----------------------------------------------------------------- general (rectangular) class

RECT_CASES = [
    # (q, b1, b, r, T): odd sizes, one-element blocks, tall and wide, several tiles and ragged tails
    (2, 3, 4, 5, 7), (5, 1, 2, 4, 65), (1, 4, 2, 3, 3), (3, 20, 17, 6, 130), (7, 5, 33, 9, 70),
    (4, 64, 64, 4, 257), (4, 96, 32, 16, 129), (16, 16, 16, 16, 100), (32, 32, 32, 32, 65),
    (4, 256, 256, 4, 200), (256, 4, 4, 256, 131), (8, 48, 80, 24, 90), (3, 5, 7, 2, 33), (2, 8, 6, 4, 50),
    # bf16 with b1 and b multiples of 64: stage 1 on the tensor cores (128- and 64-wide output tiles, K = 64..1024)
    (2, 128, 192, 3, 300), (3, 64, 128, 5, 1), (4, 1024, 1024, 4, 140), (1, 320, 448, 2, 513), (6, 192, 64, 7, 128),
    # L's blocks between 4 x 4 and 16 x 16: the shared-memory stage-2 kernel
    (16, 256, 256, 16, 70), (12, 8, 64, 5, 40), (5, 64, 128, 16, 33),
    # the TMA-fed stage 2 at its edges: one token, a ragged tile, many slabs
    (2, 64, 256, 3, 1), (4, 64, 256, 4, 17), (3, 64, 512, 4, 20011),
]


def _rect_inputs(q, b1, b, r, T, dtype, seed):
    rng = np.random.default_rng(seed)

    def draw(shape, std):
        return round_to_storage(rng.standard_normal(shape, dtype=np.float32) * np.float32(std), dtype)

    return {"x": draw((T, q * b1), 1.0), "R": draw((q, b, b1), 1.0 / np.sqrt(b1)),
            "L": draw((b, r, q), 1.0 / np.sqrt(q))}


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("q,b1,b,r,T", RECT_CASES)
def test_rect_fwd(P, impl, q, b1, b, r, T, dtype):
    import torch
    code = _code(P, dtype)
    if impl == "staged" and not (dtype == "bf16" and b1 % 64 == 0 and b % 64 == 0):
        pytest.skip("the CUDA-core kernels already serve this case under the automatic choice")
    d = _rect_inputs(q, b1, b, r, T, dtype, seed=q * 1000003 + b1 * 1009 + b * 31 + r)
    x, L, R = (to_device(d[k], dtype) for k in ("x", "L", "R"))
    yf, y = _guarded((T, r * b), _tdtype(dtype))
    ws = P.Workspace(P.monarch_rect_workspace_bytes(T, q, b1, b, r, code))
    P.monarch_rect_fwd(x, L, R, y, T, q, b1, b, r, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    assert_close(to_host64(y), O.rect_fwd(d["x"], d["L"], d["R"]), dtype, "rect y")
    _check_guard(yf, "rect y")


RECT_BWD_CASES = [
    (2, 3, 4, 5, 7), (5, 1, 2, 4, 65), (3, 20, 17, 6, 130), (7, 5, 33, 9, 70), (4, 64, 64, 4, 257),
    (4, 96, 32, 16, 129), (16, 16, 16, 16, 100), (4, 256, 256, 4, 200), (256, 4, 4, 256, 131), (8, 48, 80, 24, 90),
    (2, 128, 192, 3, 300), (4, 64, 256, 4, 17), (3, 64, 512, 4, 1500), (2, 192, 128, 3, 300), (4, 1024, 1024, 4, 140),
    (1, 128, 384, 2, 77),
]


def _instances(a):
    """Gradient tensor -> the problem instances the normwise error is taken over: its blocks, or the whole tensor
    when a block has fewer than 64 entries (a 2 x 1 block is a componentwise comparison, which sums with
    cancellation do not pass even in exact fp32 arithmetic)."""
    a = np.asarray(a)
    return a if a[0].size >= 64 else a.reshape(1, -1)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("q,b1,b,r,T", RECT_BWD_CASES)
def test_rect_bwd(P, q, b1, b, r, T, dtype):
    import torch
    code = _code(P, dtype)
    d = _rect_inputs(q, b1, b, r, T, dtype, seed=7 + q * 1000003 + b1 * 1009 + b * 31 + r)
    rng = np.random.default_rng(T + q)
    d["dy"] = round_to_storage(rng.standard_normal((T, r * b), dtype=np.float32), dtype)
    x, dy, L, R = (to_device(d[k], dtype) for k in ("x", "dy", "L", "R"))
    dxf, dx = _guarded((T, q * b1), _tdtype(dtype))
    dLf, dL = _guarded((b, r, q), torch.float32)
    dRf, dR = _guarded((q, b, b1), torch.float32)
    ws = P.Workspace(P.monarch_rect_bwd_workspace_bytes(T, q, b1, b, r, code))
    P.monarch_rect_bwd(x, dy, L, R, dx, dL, dR, 0, T, q, b1, b, r, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    ref = O.rect_bwd(d["x"], d["dy"], d["L"], d["R"])
    assert_close(to_host64(dx), ref["dx"], dtype, "rect dx")
    assert_close(_instances(to_host64(dL)), _instances(ref["dL"]), dtype, "rect dL")
    assert_close(_instances(to_host64(dR)), _instances(ref["dR"]), dtype, "rect dR")
    for flat, what in ((dxf, "dx"), (dLf, "dL"), (dRf, "dR")):
        _check_guard(flat, f"rect {what}")
    # second call: accumulate, with the intermediate a forward call left in its workspace
    ws_f = P.Workspace(P.monarch_rect_workspace_bytes(T, q, b1, b, r, code))
    y = torch.empty(T, r * b, dtype=_tdtype(dtype), device="cuda")
    P.monarch_rect_fwd(x, L, R, y, T, q, b1, b, r, ws_f)
    dx.fill_(float("nan"))
    P.monarch_rect_bwd(x, dy, L, R, dx, dL, dR, 1, T, q, b1, b, r, ws, fwd_workspace=ws_f)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0 and P.monarch_last_device_status(ws_f) == 0
    assert_close(to_host64(dx), ref["dx"], dtype, "rect dx (saved u)")
    assert_close(_instances(to_host64(dL)), _instances(2 * ref["dL"]), dtype, "rect dL accumulate")
    assert_close(_instances(to_host64(dR)), _instances(2 * ref["dR"]), dtype, "rect dR accumulate")


# (q, b1, b2, b3, r, T): b3 a multiple of b2, b2 a multiple of b3, neither; tiny, ragged and tensor-core sizes
RECTW_CASES = [
    (3, 2, 2, 4, 2, 7), (2, 3, 4, 2, 3, 65), (2, 2, 3, 5, 2, 130), (3, 1, 5, 3, 2, 70), (2, 4, 2, 6, 1, 33),
    (4, 64, 64, 256, 2, 257), (4, 128, 512, 256, 4, 300), (3, 20, 17, 34, 6, 129), (5, 24, 40, 8, 3, 200),
    (4, 64, 96, 160, 2, 140), (2, 48, 80, 48, 5, 90), (4, 256, 256, 256, 4, 200), (4, 1024, 512, 1024, 2, 150),
    (4, 64, 1024, 256, 3, 131),
]


def _rectw_inputs(q, b1, b2, b3, r, T, dtype, seed):
    rng = np.random.default_rng(seed)

    def draw(shape, std):
        return round_to_storage(rng.standard_normal(shape, dtype=np.float32) * np.float32(std), dtype)

    terms = q * max(1, b2 // b3)                          # entries that meet in one output element
    return {"x": draw((T, q * b1), 1.0), "R": draw((q, b2, b1), 1.0 / np.sqrt(b1)),
            "L": draw((r, q, max(b2, b3)), 1.0 / np.sqrt(terms)), "dy": draw((T, r * b3), 1.0)}


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("q,b1,b2,b3,r,T", RECTW_CASES)
def test_rect_wrapped_fwd_bwd(P, q, b1, b2, b3, r, T, dtype):
    """The rectangular class with wrapped-diagonal blocks (b2 != b3): forward, then dx, dL, dR (overwrite, then
    accumulate) against the oracle, over sizes that take the re-labelled fast path in both directions and sizes that
    take the general kernels."""
    import torch
    code = _code(P, dtype)
    if dtype == "bf16" and min(q * b1, r * b3) < 64:
        pytest.skip("token rows of fewer than 64 elements make the normwise bf16 comparison a componentwise one; "
                    "these index-arithmetic cases run in fp32, at 1e-5")
    d = _rectw_inputs(q, b1, b2, b3, r, T, dtype, seed=11 + q * 1000003 + b1 * 1009 + b2 * 31 + b3)
    x, dy, L, R = (to_device(d[k], dtype) for k in ("x", "dy", "L", "R"))
    bmax = max(b2, b3)
    yf, y = _guarded((T, r * b3), _tdtype(dtype))
    ws = P.Workspace(P.monarch_rectw_workspace_bytes(T, q, b1, b2, b3, r, code))
    P.monarch_rectw_fwd(x, L, R, y, T, q, b1, b2, b3, r, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    assert_close(to_host64(y), O.rectw_fwd(d["x"], d["L"], d["R"], b3), dtype, "wrapped y")
    _check_guard(yf, "wrapped y")
    dxf, dx = _guarded((T, q * b1), _tdtype(dtype))
    dLf, dL = _guarded((r, q, bmax), torch.float32)
    dRf, dR = _guarded((q, b2, b1), torch.float32)
    wsb = P.Workspace(P.monarch_rectw_bwd_workspace_bytes(T, q, b1, b2, b3, r, code))
    P.monarch_rectw_bwd(x, dy, L, R, dx, dL, dR, 0, T, q, b1, b2, b3, r, wsb)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(wsb) == 0
    ref = O.rectw_bwd(d["x"], d["dy"], d["L"], d["R"], b3)
    assert_close(to_host64(dx), ref["dx"], dtype, "wrapped dx")
    # a block of L has max(b2, b3) entries; all of dL is one instance when that is small (reading S13)
    assert_close(_instances(to_host64(dL).reshape(r * q, bmax)), _instances(ref["dL"].reshape(r * q, bmax)), dtype, "wrapped dL")
    assert_close(_instances(to_host64(dR)), _instances(ref["dR"]), dtype, "wrapped dR")
    for flat, what in ((dxf, "dx"), (dLf, "dL"), (dRf, "dR")):
        _check_guard(flat, f"wrapped {what}")
    P.monarch_rectw_bwd(x, dy, L, R, dx, dL, dR, 1, T, q, b1, b2, b3, r, wsb)
    torch.cuda.synchronize()
    assert_close(_instances(to_host64(dL).reshape(r * q, bmax)), _instances(2 * ref["dL"].reshape(r * q, bmax)), dtype,
                 "wrapped dL accumulate")
    assert_close(_instances(to_host64(dR)), _instances(2 * ref["dR"]), dtype, "wrapped dR accumulate")


def test_rect_wrapped_equal_sizes_is_the_diagonal_case(P):
    """b2 = b3: the wrapped call equals monarch_rect_fwd on the transposed weight layout, bit for bit."""
    import torch
    q, b1, b, r, T, dtype = 4, 128, 256, 3, 300, "bf16"
    d = _rectw_inputs(q, b1, b, b, r, T, dtype, seed=99)
    x, L, R = (to_device(d[k], dtype) for k in ("x", "L", "R"))
    Lp = L.permute(2, 0, 1).contiguous()
    y1 = torch.empty(T, r * b, dtype=torch.bfloat16, device="cuda")
    y2 = torch.empty_like(y1)
    P.monarch_rectw_fwd(x, L, R, y1, T, q, b1, b, b, r, P.Workspace(P.monarch_rectw_workspace_bytes(T, q, b1, b, b, r, P.BF16)))
    P.monarch_rect_fwd(x, Lp, R, y2, T, q, b1, b, r, P.Workspace(P.monarch_rect_workspace_bytes(T, q, b1, b, r, P.BF16)))
    torch.cuda.synchronize()
    assert torch.equal(y1, y2)


def test_rect_square_case_equals_monarch_fwd(P):
    """q = b1 = b = r = m is Definition 3.1: both entry points see the same tensors."""
    import torch
    m, T = 32, 130
    n = m * m
    d = _small_inputs(m, T, "f32", seed=5)
    x, L, R = (to_device(d[k], "f32") for k in ("x", "L", "R"))
    y1, y2 = torch.empty_like(x), torch.empty_like(x)
    ws = P.Workspace(max(P.monarch_workspace_bytes(P.OP_FWD, T, n, m, P.F32),
                         P.monarch_rect_workspace_bytes(T, m, m, m, m, P.F32)))
    P.monarch_fwd(x, L, R, y1, T, n, m, ws)
    P.monarch_rect_fwd(x, L, R, y2, T, m, m, m, m, ws)
    torch.cuda.synchronize()
    assert_close(to_host64(y2), to_host64(y1), "f32", "rect vs square")
    assert_close(to_host64(y2), O.fwd(d["x"], d["L"], d["R"]), "f32", "rect vs oracle")


def test_workload_rect_wrapped(P):
    """The measured case of the wrapped-diagonal class (workload 9: R four 1024 x 1024 blocks, L a 2 x 4 grid of
    2048 x 1024 wrapped diagonals, 8192 tokens) at full size, in the configuration the benchmark times: both edge rows
    and a random interior row of every 64-token tile against the oracle, finiteness of the whole output, and the
    adjoint identity <dy, y> = <dx, x> with the Euler identities <dL, L> = <dR, R> = <dy, y> on the device results."""
    import torch
    from paper_2204_00595_b200.inputs import make_rectw_inputs
    d = make_rectw_inputs()
    q, b1, b2, b3, r, T = d["q"], d["b1"], d["b2"], d["b3"], d["r"], d["tokens"]
    x, L, R = (to_device(d[k], "bf16") for k in ("x", "L", "R"))
    y = torch.full((T, r * b3), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = P.Workspace(P.monarch_rectw_workspace_bytes(T, q, b1, b2, b3, r, P.BF16))
    P.monarch_rectw_fwd(x, L, R, y, T, q, b1, b2, b3, r, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    assert bool(torch.isfinite(y.float()).all())
    rows = _tile_rows(T, 9)
    ref = O.rectw_fwd(d["x"][rows], d["L"], d["R"], b3)
    assert_close(to_host64(y[torch.from_numpy(rows).cuda()]), ref, "bf16", "wrapped workload y")
    dy = torch.randn(T, r * b3, device="cuda", generator=torch.Generator("cuda").manual_seed(9)).bfloat16()
    dx = torch.empty_like(x)
    dL = torch.empty(L.shape, dtype=torch.float32, device="cuda")
    dR = torch.empty(R.shape, dtype=torch.float32, device="cuda")
    wsb = P.Workspace(P.monarch_rectw_bwd_workspace_bytes(T, q, b1, b2, b3, r, P.BF16))
    P.monarch_rectw_bwd(x, dy, L, R, dx, dL, dR, 0, T, q, b1, b2, b3, r, wsb)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(wsb) == 0
    refb = O.rectw_bwd(d["x"][rows], to_host64(dy)[rows], d["L"], d["R"], b3)
    assert_close(to_host64(dx[torch.from_numpy(rows).cuda()]), refb["dx"], "bf16", "wrapped workload dx")
    dot = lambda a, b: float((a.double() * b.double()).sum())
    # sums of T*r*b3 products of unit-variance factors: the identities hold to the bf16 rounding of y, dx and u
    s_y, tol = dot(dy, y), 2e-2 * float(np.sqrt(T * r * b3))
    for what, v in (("<dx, x>", dot(dx, x)), ("<dL, L>", dot(dL, L)), ("<dR, R>", dot(dR, R))):
        assert abs(v - s_y) <= tol, (what, v, s_y)


def test_workload_rect(P, impl):
    """The measured case of the general class (four 1024 x 1024 blocks, 8192 tokens) at full size: sampled
    token rows against the oracle, and the stage-2-is-identity special case on all rows."""
    import torch
    from paper_2204_00595_b200.inputs import make_rect_inputs
    d = make_rect_inputs()
    q, b1, b, r, T = d["q"], d["b1"], d["b"], d["r"], d["tokens"]
    x, L, R = (to_device(d[k], "bf16") for k in ("x", "L", "R"))
    y = torch.full((T, r * b), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = P.Workspace(P.monarch_rect_workspace_bytes(T, q, b1, b, r, P.BF16))
    P.monarch_rect_fwd(x, L, R, y, T, q, b1, b, r, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    assert bool(torch.isfinite(y.float()).all())
    rows = _sample_tokens(T, 96, 6)
    ref = O.rect_fwd(d["x"][rows], d["L"], d["R"])
    assert_close(to_host64(y[torch.from_numpy(rows).cuda()]), ref, "bf16", "rect workload y")
    # L's blocks = identity (r = q): y = u = blockdiag(R) x, one bf16 rounding more than a plain block product
    Li = to_device(np.broadcast_to(np.eye(q, dtype=np.float32), (b, q, q)).copy(), "bf16")
    P.monarch_rect_fwd(x, Li, R, y, T, q, b1, b, r, ws)
    torch.cuda.synchronize()
    ref = np.einsum("kji,tki->tkj", d["R"].astype(np.float64), d["x"][rows].astype(np.float64).reshape(-1, q, b1))
    assert_close(to_host64(y[torch.from_numpy(rows).cuda()]), ref.reshape(len(rows), q * b), "bf16", "rect identity L")


def test_workload_rect_bwd(P, impl):
    """Backward of the measured case at full size, in the configuration the benchmark times (the forward's
    intermediate reused): dx on sampled token rows against the oracle; the weight gradients through the Euler
    and adjoint identities <dL, L> = <dR, R> = <dx, x> = <dy, y> evaluated on the device results."""
    import torch
    from paper_2204_00595_b200.inputs import make_rect_inputs
    d = make_rect_inputs()
    q, b1, b, r, T = d["q"], d["b1"], d["b"], d["r"], d["tokens"]
    rng = np.random.default_rng(606)
    dy_h = round_to_storage(rng.standard_normal((T, r * b), dtype=np.float32), "bf16")
    x, L, R, dy = (to_device(a, "bf16") for a in (d["x"], d["L"], d["R"], dy_h))
    y = torch.empty(T, r * b, dtype=torch.bfloat16, device="cuda")
    dx = torch.full((T, q * b1), float("nan"), dtype=torch.bfloat16, device="cuda")
    dL = torch.full((b, r, q), float("nan"), dtype=torch.float32, device="cuda")
    dR = torch.full((q, b, b1), float("nan"), dtype=torch.float32, device="cuda")
    ws_f = P.Workspace(P.monarch_rect_workspace_bytes(T, q, b1, b, r, P.BF16))
    ws_b = P.Workspace(P.monarch_rect_bwd_workspace_bytes(T, q, b1, b, r, P.BF16))
    P.monarch_rect_fwd(x, L, R, y, T, q, b1, b, r, ws_f)
    P.monarch_rect_bwd(x, dy, L, R, dx, dL, dR, 0, T, q, b1, b, r, ws_b, fwd_workspace=ws_f)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws_b) == 0 and P.monarch_last_device_status(ws_f) == 0
    rows = _sample_tokens(T, 64, 66)
    ref = O.rect_bwd(d["x"][rows], dy_h[rows], d["L"], d["R"])
    dxh = to_host64(dx)
    assert np.isfinite(dxh).all()
    assert_close(dxh[rows], ref["dx"], "bf16", "rect workload dx")
    s = float(np.sum(dy_h.astype(np.float64) * to_host64(y)))
    tol = 2e-2 * float(np.sqrt(T * r * b))
    assert abs(float(np.sum(dxh * d["x"])) - s) <= tol
    assert abs(float(np.sum(to_host64(dL) * d["L"])) - s) <= tol
    assert abs(float(np.sum(to_host64(dR) * d["R"])) - s) <= tol


def test_rect_arguments(P):
    import torch
    x = torch.zeros(4, 64, device="cuda")
    ws = P.Workspace(1 << 16)
    assert P.monarch_rect_workspace_bytes(4, 0, 8, 8, 8, P.F32) == 0
    assert P.monarch_rect_workspace_bytes(4, 8, 8, 8, 1 << 20, P.F32) == 0
    with pytest.raises(P.MonarchError):
        P.monarch_rect_fwd(x, x, x, x.clone(), 4, 8, 8, 8, -1, ws)
    y = torch.full((1, 8), 3.0, device="cuda")
    P.monarch_rect_fwd(x, x, x, y, 0, 2, 4, 4, 2, ws)            # zero tokens: nothing written
    torch.cuda.synchronize()
    assert float(y.min()) == 3.0


# ----------------------------------------------------------------- complex factors (planar tensors)

def _planar(z, dtype):
    """complex array -> float32 [2, ...] planes rounded to the storage dtype (and the complex value they hold)."""
    planes = np.stack([round_to_storage(z.real.astype(np.float32), dtype),
                       round_to_storage(z.imag.astype(np.float32), dtype)])
    return planes, planes[0].astype(np.float64) + 1j * planes[1].astype(np.float64)


@pytest.mark.parametrize("adjoint", [0, 1])
@pytest.mark.parametrize("m,T,dtype", [(16, 37, "f32"), (32, 130, "f32"), (32, 65, "bf16"), (64, 129, "bf16"),
                                       (128, 70, "bf16")])
def test_cplx_fwd(P, impl, m, T, dtype, adjoint):
    import torch
    code = _code(P, dtype)
    _skip_if_same_family(P, impl, P.OP_CPLX, m, code)
    n = m * m
    rng = np.random.default_rng(800 + m + T)
    xp, xc = _planar(rng.standard_normal((T, n)) + 1j * rng.standard_normal((T, n)), dtype)
    s = 1.0 / np.sqrt(2 * m)
    Lp, Lc = _planar(s * (rng.standard_normal((m, m, m)) + 1j * rng.standard_normal((m, m, m))), dtype)
    Rp, Rc = _planar(s * (rng.standard_normal((m, m, m)) + 1j * rng.standard_normal((m, m, m))), dtype)
    x, L, R = to_device(xp, dtype), to_device(Lp, dtype), to_device(Rp, dtype)
    yf, y = _guarded((2, T, n), _tdtype(dtype))
    ws = P.Workspace(P.monarch_workspace_bytes(P.OP_CPLX, T, n, m, code))
    P.monarch_cplx_fwd(x, L, R, y, adjoint, T, n, m, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    ref = O.cplx_fwd(xc, Lc, Rc, adjoint=bool(adjoint))
    yh = to_host64(y)
    # a problem instance is a token's complex row: compare re and im side by side
    assert_close(np.concatenate([yh[0], yh[1]], axis=1), np.concatenate([ref.real, ref.imag], axis=1), dtype,
                 f"complex y adjoint={adjoint}")
    _check_guard(yf, "complex y")


def test_cplx_dft_closed_form(P):
    """Section 3.2: with the Cooley-Tukey factors the multiply is the DFT of the permuted input; numpy.fft is
    the reference, independent of the oracle's loops."""
    import torch
    m, T = 16, 33
    n = m * m
    rng = np.random.default_rng(816)
    Lc, Rc = O.dft_factors(m)
    Lp, _ = _planar(Lc, "f32")
    Rp, _ = _planar(Rc, "f32")
    xp, xc = _planar(rng.standard_normal((T, n)) + 1j * rng.standard_normal((T, n)), "f32")
    xperm = xc.reshape(T, m, m).transpose(0, 2, 1).reshape(T, n)                   # P x
    xpp, _ = _planar(xperm, "f32")
    y = torch.empty(2, T, n, device="cuda")
    ws = P.Workspace(P.monarch_workspace_bytes(P.OP_CPLX, T, n, m, P.F32))
    P.monarch_cplx_fwd(to_device(xpp, "f32"), to_device(Lp, "f32"), to_device(Rp, "f32"), y, 0, T, n, m, ws)
    torch.cuda.synchronize()
    ref = np.fft.fft(xc, axis=1)
    yh = to_host64(y)
    assert_close(np.concatenate([yh[0], yh[1]], axis=1), np.concatenate([ref.real, ref.imag], axis=1), "f32",
                 "DFT")


# ----------------------------------------------------------------- dense <-> factors (Eq. 2, Algorithm 1)

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("m", [16, 32, 64])
def test_dense_from_factors(P, m, dtype):
    import torch
    n = m * m
    d = _small_inputs(m, 1, dtype, seed=40 + m)
    L, R = to_device(d["L"], dtype), to_device(d["R"], dtype)
    Mf, M = _guarded((n, n), _tdtype(dtype))
    P.monarch_dense(L, R, M, n, m)
    torch.cuda.synchronize()
    assert_close(to_host64(M), O.dense(d["L"], d["R"]), dtype, "dense")
    _check_guard(Mf, "dense")


def _project_gpu(P, A32, m, dtype):
    import torch
    n = m * m
    A = to_device(A32, dtype)
    Lf, L = _guarded((m, m, m), _tdtype(dtype))
    Rf, R = _guarded((m, m, m), _tdtype(dtype))
    rot = torch.zeros(1, dtype=torch.int64, device="cuda")
    P.monarch_project(A, L, R, n, m, rotation_count=rot)
    torch.cuda.synchronize()
    _check_guard(Lf, "project L")
    _check_guard(Rf, "project R")
    assert int(rot.item()) > 0
    return to_host64(L), to_host64(R)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("m", [16, 32, 64])
def test_project_recovers_monarch_and_planted(P, m, dtype):
    """Section 3.3: a Monarch input is recovered; with small noise added the slices keep a clear leading
    singular value, so the rank-1 pieces are well conditioned and must match the oracle's (numpy SVD)."""
    rng = np.random.default_rng(600 + m)
    d = _small_inputs(m, 1, dtype, seed=50 + m)
    A = O.dense(d["L"], d["R"])
    A32 = round_to_storage(A.astype(np.float32), dtype)
    Lg, Rg = _project_gpu(P, A32, m, dtype)
    assert_close(O.dense(Lg, Rg), A32.astype(np.float64), dtype, "project(monarch)")
    noisy = round_to_storage((A + 0.02 / m * rng.standard_normal(A.shape)).astype(np.float32), dtype)
    Lg, Rg = _project_gpu(P, noisy, m, dtype)
    Lo, Ro = O.project(noisy.astype(np.float64), m)
    assert_close(O.dense(Lg, Rg), O.dense(Lo, Ro), dtype, "project(planted)")


@pytest.mark.parametrize("m", [16, 64])
def test_project_generic_is_optimal(P, m):
    """Theorem 1: the residual of the projection equals the discarded spectrum of the slices - a criterion
    that does not depend on the gap between the first two singular values."""
    rng = np.random.default_rng(700 + m)
    n = m * m
    A32 = rng.standard_normal((n, n), dtype=np.float32)
    Lg, Rg = _project_gpu(P, A32, m, "f32")
    A = A32.astype(np.float64)
    res = float(np.sum((A - O.dense(Lg, Rg)) ** 2))
    sv = np.linalg.svd(A.reshape(m, m, m, m).transpose(1, 2, 0, 3).reshape(m * m, m, m), compute_uv=False)
    tail = float(np.sum(sv[:, 1:] ** 2))
    assert tail * (1 - 1e-9) <= res <= tail * (1 + 1e-5)


def test_project_m128_sampled_slices(P):
    rng = np.random.default_rng(728)
    m = 128
    n = m * m
    A32 = rng.standard_normal((n, n), dtype=np.float32)
    Lg, Rg = _project_gpu(P, A32, m, "f32")
    A4 = A32.reshape(m, m, m, m)                           # [l, j, k, i]
    for j, k in [(0, 0), (5, 127), (127, 3), (64, 64), (17, 90)]:
        S = A4[:, j, k, :].astype(np.float64)
        sv = np.linalg.svd(S, compute_uv=False)
        res = float(np.sum((S - np.outer(Lg[j, :, k], Rg[k, j, :])) ** 2))
        tail = float(np.sum(sv[1:] ** 2))
        assert tail * (1 - 1e-9) <= res <= tail * (1 + 1e-5)


# ----------------------------------------------------------------- the five workloads

def _sample_tokens(T, count, seed):
    rng = np.random.default_rng(seed)
    idx = set(rng.choice(T, size=min(count, T), replace=False).tolist())
    idx.update({0, 1, T // 2, T - 2, T - 1} & set(range(T)))
    return np.array(sorted(idx))


def _tile_rows(T, seed, tile=64):
    """Both edges and one random interior row of every 64-token tile (the finest token tiling any kernel uses;
    coarser tiles and every CTA / team residue are unions of these)."""
    rng = np.random.default_rng(seed)
    idx = set()
    for t0 in range(0, T, tile):
        t1 = min(t0 + tile, T)
        idx.update({t0, t1 - 1, int(rng.integers(t0, t1))})
    return np.array(sorted(idx))


@pytest.mark.parametrize("cfg", [1, 2, 3, 4])
def test_workload_fwd_bwd(P, impl, cfg):
    """Full-size workloads 1-4: every row of y and dx and all of dL and dR against the oracle, plus the
    adjoint and Euler identities evaluated on the device results."""
    import torch
    c = CONFIGS[cfg]
    code = _code(P, c.dtype)
    _skip_if_same_family(P, impl, P.OP_FWD, c.m, code)
    d = make_inputs(cfg)
    m, n, T = c.m, c.n, c.tokens
    x, L, R = (to_device(d[k], c.dtype) for k in ("x", "L", "R"))
    y = torch.full_like(x, float("nan"))
    ops = [P.OP_FWD] + ([P.OP_BWD_DX, P.OP_BWD_DW] if "bwd_dx" in c.ops else [])
    ws = P.Workspace(max(P.monarch_workspace_bytes(op, T, n, m, code) for op in ops))
    P.monarch_fwd(x, L, R, y, T, n, m, ws)
    torch.cuda.synchronize()
    rows = np.arange(T)
    ref_y = O.fwd(d["x"], d["L"], d["R"])
    yh = to_host64(y)
    assert np.isfinite(yh).all()
    assert_close(yh, ref_y, c.dtype, f"cfg{cfg} y")
    if "bwd_dx" not in c.ops:
        assert P.monarch_last_device_status(ws) == 0
        return
    dy = to_device(d["dy"], c.dtype)
    dx = torch.full_like(x, float("nan"))
    dL = torch.full((m, m, m), float("nan"), dtype=torch.float32, device="cuda")
    dR = torch.full_like(dL, float("nan"))
    P.monarch_bwd_dx(dy, L, R, dx, T, n, m, ws)
    P.monarch_bwd_dw(x, dy, L, R, dL, dR, 0, T, n, m, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    ref = O.bwd(d["x"], d["dy"], d["L"], d["R"])
    dxh, dLh, dRh = to_host64(dx), to_host64(dL), to_host64(dR)
    assert_close(dxh[rows], ref["dx"][rows], c.dtype, f"cfg{cfg} dx")
    assert_close(dLh, ref["dL"], c.dtype, f"cfg{cfg} dL")
    assert_close(dRh, ref["dR"], c.dtype, f"cfg{cfg} dR")
    # identities that hold at any size, from device results only (fp64 sums on the host)
    s = float(np.sum(d["dy"].astype(np.float64) * yh))
    scale = float(np.sqrt(T * n))            # size of a random-sign sum of T*n unit terms
    tol = 2e-2 * scale
    assert abs(float(np.sum(dxh * d["x"])) - s) <= tol
    assert abs(float(np.sum(dLh * d["L"])) - s) <= tol
    assert abs(float(np.sum(dRh * d["R"])) - s) <= tol
    # the one-call backward on the intermediate the forward call left in its workspace (the launch
    # configuration the benchmark times)
    ws_b = P.Workspace(P.monarch_workspace_bytes(P.OP_BWD, T, n, m, code))
    dx.fill_(float("nan")); dL.fill_(float("nan")); dR.fill_(float("nan"))
    P.monarch_fwd(x, L, R, y, T, n, m, ws)
    P.monarch_bwd(x, dy, L, R, dx, dL, dR, 0, T, n, m, ws_b, fwd_workspace=ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws_b) == 0
    assert_close(to_host64(dx)[rows], ref["dx"][rows], c.dtype, f"cfg{cfg} dx (one call)")
    assert_close(to_host64(dL), ref["dL"], c.dtype, f"cfg{cfg} dL (one call)")
    assert_close(to_host64(dR), ref["dR"], c.dtype, f"cfg{cfg} dR (one call)")


def test_workload_mlp(P, impl):
    import torch
    c = CONFIGS[5]
    code = _code(P, c.dtype)
    _skip_if_same_family(P, impl, P.OP_MLP_FWD, c.m, code)
    d = make_inputs(5)
    m, n, T = c.m, c.n, c.tokens
    t = {k: to_device(d[k], c.dtype) for k in ("x", "L", "R", "b1", "L2", "R2", "b2")}
    y = torch.full_like(t["x"], float("nan"))
    ws = P.Workspace(P.monarch_workspace_bytes(P.OP_MLP_FWD, T, n, m, code))
    P.monarch_mlp_fwd(t["x"], t["L"], t["R"], t["b1"], t["L2"], t["R2"], t["b2"], y, T, n, m, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    rows = _tile_rows(T, 5)                      # 3 rows of each of the 512 tiles
    ref = O.mlp_fwd(d["x"][rows], d["L"], d["R"], d["b1"], d["L2"], d["R2"], d["b2"])
    yh = to_host64(y[torch.from_numpy(rows).cuda()])
    assert bool(torch.isfinite(y.float()).all())
    assert_close(yh, ref, c.dtype, "cfg5 mlp y")


def test_workload_mlp_bwd(P, impl):
    """Backward of the feed-forward block on workload 5's tensors: every gradient against the oracle on a
    ragged slice of the tokens, then the full token count with dx on sampled rows, db2 against its
    definition and the Euler identities of the two bilinear maps evaluated on the device results."""
    import torch
    c = CONFIGS[5]
    code = _code(P, c.dtype)
    _skip_if_same_family(P, impl, P.OP_MLP_BWD, c.m, code)
    d = make_inputs(5, with_dy=True)
    m, n, T = c.m, c.n, c.tokens
    t = {k: to_device(d[k], c.dtype) for k in ("x", "dy", "L", "R", "b1", "L2", "R2", "b2")}
    ws = P.Workspace(P.monarch_workspace_bytes(P.OP_MLP_BWD, T, n, m, code))
    # (1) a slice the oracle finishes in seconds: 17 tiles and a ragged tail
    Ts = 1100
    ts = {k: (v[:Ts].contiguous() if k in ("x", "dy") else v) for k, v in t.items()}
    bufs = _mlp_bwd_buffers(m, Ts, c.dtype)
    _call_mlp_bwd(P, ts, bufs, 0, Ts, n, m, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    ref = O.mlp_bwd(d["x"][:Ts], d["dy"][:Ts], d["L"], d["R"], d["b1"], d["L2"], d["R2"])
    assert_close(to_host64(bufs["dx"][1]), ref["dx"], c.dtype, "cfg5 slice dx")
    _assert_mlp_grads(bufs, ref, c.dtype, "cfg5 slice")
    # (2) all tokens
    bufs = _mlp_bwd_buffers(m, T, c.dtype)
    _call_mlp_bwd(P, t, bufs, 0, T, n, m, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    rows = _tile_rows(T, 55)
    ref = O.mlp_bwd(d["x"][rows], d["dy"][rows], d["L"], d["R"], d["b1"], d["L2"], d["R2"])
    dxh = to_host64(bufs["dx"][1])
    assert np.isfinite(dxh).all()
    assert_close(dxh[rows], ref["dx"], c.dtype, "cfg5 dx")
    g = {k: to_host64(bufs[k][1]) for k in MLP_GRADS}
    assert_close(g["db2"][None, :], d["dy"].astype(np.float64).sum(0)[None, :], c.dtype, "cfg5 db2")
    # y - b2 is bilinear in (L2, R2) and a - b1 in (L1, R1):
    #   <dL2, L2> = <dR2, R2> = <dy, y - b2>,   <dL1, L1> = <dR1, R1> = <dx, x>
    y = torch.empty_like(t["x"])
    ws_f = P.Workspace(P.monarch_workspace_bytes(P.OP_MLP_FWD, T, n, m, code))
    P.monarch_mlp_fwd(t["x"], t["L"], t["R"], t["b1"], t["L2"], t["R2"], t["b2"], y, T, n, m, ws_f)
    torch.cuda.synchronize()
    s2 = float(np.sum(d["dy"].astype(np.float64) * (to_host64(y) - d["b2"].astype(np.float64))))
    tol = 2e-2 * float(np.sqrt(T * n))
    assert abs(float(np.sum(g["dL2"] * d["L2"])) - s2) <= tol
    assert abs(float(np.sum(g["dR2"] * d["R2"])) - s2) <= tol
    s1 = float(np.sum(dxh * d["x"]))
    assert abs(float(np.sum(g["dL1"] * d["L"])) - s1) <= tol
    assert abs(float(np.sum(g["dR1"] * d["R"])) - s1) <= tol


# ----------------------------------------------------------------- a bounded wait that runs out

def test_bounded_wait_runs_out_and_the_workspace_recovers(P):
    """One operand load of the m = 128 forward is left out on the host side (nothing faults): the thread block
    that waits for it gives up after the 5 ms limit set here, the call returns, the status word reads
    MONARCH_ERR_TIMEOUT once, and after monarch_workspace_init the same workspace serves a correct call."""
    import time
    import torch
    m, T, dtype = 128, 129, "bf16"
    n = m * m
    d = _small_inputs(m, T, dtype, seed=4242)
    x, L, R = (to_device(d[k], dtype) for k in ("x", "L", "R"))
    y = torch.full_like(x, float("nan"))
    ws = P.Workspace(P.monarch_workspace_bytes(P.OP_FWD, T, n, m, P.BF16))
    assert P.monarch_impl_name(P.OP_FWD, m, P.BF16) == "staged-tcgen05"
    P.monarch_debug_set_wait_limit(ws, 5000)
    P.monarch_debug_skip_load(0)
    t0 = time.perf_counter()
    P.monarch_fwd(x, L, R, y, T, n, m, ws)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 5.0          # the wait ended at its limit, not at the default second
    assert P.monarch_last_device_status(ws) == 5   # MONARCH_ERR_TIMEOUT
    assert P.monarch_last_device_status(ws) == 0   # cleared on read
    P.monarch_workspace_init(ws)
    y.fill_(float("nan"))
    P.monarch_fwd(x, L, R, y, T, n, m, ws)
    torch.cuda.synchronize()
    assert P.monarch_last_device_status(ws) == 0
    assert_close(to_host64(y), O.fwd(d["x"], d["L"], d["R"]), dtype, "y after recovery")


# ----------------------------------------------------------------- the m = 64 forward on clusters of four CTAs

@pytest.mark.parametrize("T", [1, 63, 130, 257, 2500])
def test_fwd_m64_on_clusters(T):
    """The variant that keeps the permuted intermediate in distributed shared memory (selected by an environment
    variable read once per process, hence the child process) against the oracle."""
    import os
    import subprocess
    import sys
    code = f"""
import sys, numpy as np, torch
sys.path.insert(0, {os.path.dirname(os.path.dirname(os.path.abspath(__file__)))!r})
import paper_2204_00595_b200 as P
from oracle import monarch_oracle as O
from paper_2204_00595_b200.inputs import round_to_storage, to_device, to_host64
from tests.helpers import assert_close
m, n, T = 64, 4096, {T}
rng = np.random.default_rng(6400 + T)
draw = lambda shape, std: round_to_storage(rng.standard_normal(shape, dtype=np.float32) * np.float32(std), "bf16")
hx, hL, hR = draw((T, n), 1.0), draw((m, m, m), 0.125), draw((m, m, m), 0.125)
x, L, R = (to_device(a, "bf16") for a in (hx, hL, hR))
y = torch.full_like(x, float("nan"))
ws = P.Workspace(P.monarch_workspace_bytes(P.OP_FWD, T, n, m, P.BF16))
for _ in range(2):
    P.monarch_fwd(x, L, R, y, T, n, m, ws)
torch.cuda.synchronize()
assert P.monarch_last_device_status(ws) == 0
assert_close(to_host64(y), O.fwd(hx, hL, hR), "bf16", "y on clusters")
print("ok")
"""
    env = dict(os.environ, MONARCH_M64_CLUSTER="1")
    out = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "ok" in out.stdout, out.stderr[-2000:]


# ----------------------------------------------------------------- m = 128: the three-launch forward, and run-to-run bits

@pytest.mark.parametrize("T", [1, 130, 700])
def test_fwd_m128_as_three_launches(T):
    """The forward of the m = 128 chain in its three-launch form (what a device too small for the persistent launch,
    or a batch of more than 8192 tiles, gets; selected by an environment variable read once per process, hence the
    child process), and the backward reading the u' that form left behind, against the oracle."""
    import os
    import subprocess
    import sys
    code = f"""
import sys, numpy as np, torch
sys.path.insert(0, {os.path.dirname(os.path.dirname(os.path.abspath(__file__)))!r})
import paper_2204_00595_b200 as P
from oracle import monarch_oracle as O
from paper_2204_00595_b200.inputs import round_to_storage, to_device, to_host64
from tests.helpers import assert_close
m, n, T = 128, 16384, {T}
rng = np.random.default_rng(12800 + T)
draw = lambda shape, std: round_to_storage(rng.standard_normal(shape, dtype=np.float32) * np.float32(std), "bf16")
hx, hdy, hL, hR = draw((T, n), 1.0), draw((T, n), 1.0), draw((m, m, m), 0.088), draw((m, m, m), 0.088)
x, dy, L, R = (to_device(a, "bf16") for a in (hx, hdy, hL, hR))
y = torch.full_like(x, float("nan")); dx = torch.full_like(x, float("nan"))
dL = torch.full((m, m, m), float("nan"), device="cuda"); dR = torch.full((m, m, m), float("nan"), device="cuda")
ws = P.Workspace(P.monarch_workspace_bytes(P.OP_FWD, T, n, m, P.BF16))
wsb = P.Workspace(P.monarch_workspace_bytes(P.OP_BWD, T, n, m, P.BF16))
n0 = P.monarch_launch_count()
P.monarch_fwd(x, L, R, y, T, n, m, ws)
assert P.monarch_launch_count() - n0 == 3
P.monarch_bwd(x, dy, L, R, dx, dL, dR, 0, T, n, m, wsb, fwd_workspace=ws)
torch.cuda.synchronize()
assert P.monarch_last_device_status(ws) == 0 and P.monarch_last_device_status(wsb) == 0
ref = O.bwd(hx, hdy, hL, hR)
assert_close(to_host64(y), O.fwd(hx, hL, hR), "bf16", "y, three launches")
assert_close(to_host64(dx), ref["dx"], "bf16", "dx")
assert_close(to_host64(dL), ref["dL"], "bf16", "dL")
assert_close(to_host64(dR), ref["dR"], "bf16", "dR")
print("ok")
"""
    env = dict(os.environ, MONARCH_CHAIN_SPLIT="1")
    out = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "ok" in out.stdout, out.stderr[-2000:]


def test_m128_weight_gradients_have_the_same_bits_every_run(P):
    """bf16 m = 128: one thread block sums all tokens of a weight block in a fixed order, so dL and dR do not depend on
    timing - three runs from different initial contents (overwrite mode), with and without the saved u', agree bit
    for bit; accumulate = 1 from equal contents does too."""
    import torch
    m, T, dtype = 128, 700, "bf16"
    n = m * m
    d = _small_inputs(m, T, dtype, seed=128700)
    x, dy, L, R = (to_device(d[k], dtype) for k in ("x", "dy", "L", "R"))
    y = torch.empty_like(x)
    dx = torch.empty_like(x)
    ws_f = P.Workspace(P.monarch_workspace_bytes(P.OP_FWD, T, n, m, P.BF16))
    ws_b = P.Workspace(P.monarch_workspace_bytes(P.OP_BWD, T, n, m, P.BF16))
    P.monarch_fwd(x, L, R, y, T, n, m, ws_f)
    runs = []
    for fill, saved, acc in ((float("nan"), True, 0), (3.0, False, 0), (-1.0, True, 0), (0.5, True, 1), (0.5, False, 1)):
        dL = torch.full((m, m, m), fill, device="cuda")
        dR = torch.full((m, m, m), fill, device="cuda")
        P.monarch_bwd(x, dy, L, R, dx, dL, dR, acc, T, n, m, ws_b, fwd_workspace=ws_f if saved else None)
        torch.cuda.synchronize()
        assert P.monarch_last_device_status(ws_b) == 0
        runs.append((dL, dR))
    for k in (1, 2):
        assert torch.equal(runs[k][0], runs[0][0]) and torch.equal(runs[k][1], runs[0][1])
    assert torch.equal(runs[3][0], runs[4][0]) and torch.equal(runs[3][1], runs[4][1])
    ref = O.bwd(d["x"], d["dy"], d["L"], d["R"])
    assert_close(to_host64(runs[0][0]), ref["dL"], dtype, "dL")
    assert_close(to_host64(runs[3][1] - 0.5), ref["dR"], dtype, "dR accumulated onto 0.5")


@pytest.mark.parametrize("T", [1, 129, 64 * 150 + 7])
def test_bwd_m32_fixed_summation_order(P, T):
    """monarch_set_deterministic(1) at bf16 m = 32 (token reductions on the tensor cores, split over token slices):
    runs from different initial contents give the same bits through monarch_bwd and monarch_bwd_dw, both match the
    oracle, accumulate = 1 adds to what is there, and a workspace sized before the switch is refused."""
    import torch
    m, dtype, code = 32, "bf16", P.BF16
    n = m * m
    d = _small_inputs(m, T, dtype, seed=3200 + T)
    x, dy, L, R = (to_device(d[k], dtype) for k in ("x", "dy", "L", "R"))
    ref = O.bwd(d["x"], d["dy"], d["L"], d["R"])
    small = P.monarch_workspace_bytes(P.OP_BWD, T, n, m, code)
    prev = P.monarch_set_deterministic(True)
    try:
        assert P.monarch_impl_name(P.OP_BWD, m, code) == "staged-tcgen05"
        nb = P.monarch_workspace_bytes(P.OP_BWD, T, n, m, code)
        assert nb == small + (32 << 20)
        ws = P.Workspace(max(nb, P.monarch_workspace_bytes(P.OP_BWD_DW, T, n, m, code)))
        dx = torch.empty_like(x)
        runs = []
        for fill, one_call in ((float("nan"), True), (11.0, True), (-3.0, False), (0.5, False)):
            dL = torch.full((m, m, m), fill, device="cuda")
            dR = torch.full((m, m, m), fill, device="cuda")
            if one_call:
                P.monarch_bwd(x, dy, L, R, dx, dL, dR, 0, T, n, m, ws)
            else:
                P.monarch_bwd_dw(x, dy, L, R, dL, dR, 0, T, n, m, ws)
            torch.cuda.synchronize()
            assert P.monarch_last_device_status(ws) == 0
            runs.append((dL, dR))
        for dL, dR in runs[1:]:
            assert torch.equal(dL, runs[0][0]) and torch.equal(dR, runs[0][1])
        assert_close(to_host64(dx), ref["dx"], dtype, "dx")
        assert_close(to_host64(runs[0][0]), ref["dL"], dtype, "dL fixed order")
        assert_close(to_host64(runs[0][1]), ref["dR"], dtype, "dR fixed order")
        dL, dR = runs[0][0].clone(), runs[0][1].clone()
        P.monarch_bwd_dw(x, dy, L, R, dL, dR, 1, T, n, m, ws)
        torch.cuda.synchronize()
        assert_close(to_host64(dL), 2 * ref["dL"], dtype, "dL accumulate, fixed order")
        assert_close(to_host64(dR), 2 * ref["dR"], dtype, "dR accumulate, fixed order")
        with pytest.raises(P.MonarchError):
            P.monarch_bwd(x, dy, L, R, dx, dL, dR, 0, T, n, m, P.Workspace(small))
    finally:
        P.monarch_set_deterministic(prev)
    assert P.monarch_workspace_bytes(P.OP_BWD, T, n, m, code) == small


@pytest.mark.parametrize("m", [16, 32, 64])
def test_fp32_weight_gradients_have_the_same_bits_every_run(P, m):
    """fp32 runs on the CUDA-core family, whose token sums are taken slab by slab and added in slab order: dL and dR
    from different initial contents (overwrite mode) agree bit for bit, through monarch_bwd and monarch_bwd_dw."""
    import torch
    T, dtype = 333, "f32"
    n = m * m
    d = _small_inputs(m, T, dtype, seed=3300 + m)
    x, dy, L, R = (to_device(d[k], dtype) for k in ("x", "dy", "L", "R"))
    dx = torch.empty_like(x)
    ws = P.Workspace(max(P.monarch_workspace_bytes(P.OP_BWD, T, n, m, P.F32),
                         P.monarch_workspace_bytes(P.OP_BWD_DW, T, n, m, P.F32)))
    runs = []
    for fill, one_call in ((float("nan"), True), (7.0, True), (-2.0, False), (0.25, False)):
        dL = torch.full((m, m, m), fill, device="cuda")
        dR = torch.full((m, m, m), fill, device="cuda")
        if one_call:
            P.monarch_bwd(x, dy, L, R, dx, dL, dR, 0, T, n, m, ws)
        else:
            P.monarch_bwd_dw(x, dy, L, R, dL, dR, 0, T, n, m, ws)
        torch.cuda.synchronize()
        assert P.monarch_last_device_status(ws) == 0
        runs.append((dL, dR))
    assert torch.equal(runs[0][0], runs[1][0]) and torch.equal(runs[0][1], runs[1][1])
    assert torch.equal(runs[2][0], runs[3][0]) and torch.equal(runs[2][1], runs[3][1])
    ref = O.bwd(d["x"], d["dy"], d["L"], d["R"])
    for k in (0, 2):
        assert_close(to_host64(runs[k][0]), ref["dL"], dtype, "dL")
        assert_close(to_host64(runs[k][1]), ref["dR"], dtype, "dR")


def test_zero_tokens_m128_and_wrapped(P):
    """An empty batch: outputs untouched, weight gradients zeroed (overwrite) or left alone (accumulate)."""
    import torch
    m = 128
    n = m * m
    x = torch.zeros(1, n, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(m, m, m, dtype=torch.bfloat16, device="cuda")
    y = torch.full((1, n), 3.0, dtype=torch.bfloat16, device="cuda")
    g = torch.full((2, m, m, m), 5.0, dtype=torch.float32, device="cuda")
    ws = P.Workspace(max(P.monarch_workspace_bytes(P.OP_FWD, 0, n, m, P.BF16), 256))
    wsb = P.Workspace(max(P.monarch_workspace_bytes(P.OP_BWD, 0, n, m, P.BF16), 256))
    P.monarch_fwd(x, W, W.clone(), y, 0, n, m, ws)
    P.monarch_bwd(x, x.clone(), W, W.clone(), y.clone(), g[0], g[1], 1, 0, n, m, wsb)
    torch.cuda.synchronize()
    assert float(y.float().min()) == 3.0 and float(g.min()) == 5.0
    P.monarch_bwd(x, x.clone(), W, W.clone(), y.clone(), g[0], g[1], 0, 0, n, m, wsb)
    torch.cuda.synchronize()
    assert float(g.abs().max()) == 0.0
    q, b1, b2, b3, r = 2, 8, 4, 8, 3
    xr = torch.zeros(1, q * b1, device="cuda")
    R = torch.zeros(q, b2, b1, device="cuda")
    L = torch.zeros(r, q, max(b2, b3), device="cuda")
    yr = torch.full((1, r * b3), 3.0, device="cuda")
    gL, gR = torch.full(L.shape, 5.0, device="cuda"), torch.full(R.shape, 5.0, device="cuda")
    w1 = P.Workspace(max(P.monarch_rectw_workspace_bytes(0, q, b1, b2, b3, r, P.F32), 256))
    w2 = P.Workspace(max(P.monarch_rectw_bwd_workspace_bytes(0, q, b1, b2, b3, r, P.F32), 256))
    P.monarch_rectw_fwd(xr, L, R, yr, 0, q, b1, b2, b3, r, w1)
    P.monarch_rectw_bwd(xr, yr.clone(), L, R, xr.clone(), gL, gR, 0, 0, q, b1, b2, b3, r, w2)
    torch.cuda.synchronize()
    assert float(yr.min()) == 3.0 and float(gL.abs().max()) == 0.0 and float(gR.abs().max()) == 0.0
