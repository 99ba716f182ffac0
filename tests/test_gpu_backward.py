"""GPU parity of mxnorm_bwd (through the C ABI) against the binary64 oracle."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2603_13180_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_13180_b200 import binding as b
    return b


def bf16_ulp(v64):
    a = np.abs(v64)
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -126)))
    return 2.0 ** (e - 7)


def run_bwd(binding, x_bits, g_bits, gain_bits, rms, fp32_out, want_dgain=True):
    T, D = x_bits.shape
    x = wl.from_bits(x_bits).cuda()
    g = wl.from_bits(g_bits).cuda()
    gain = None if gain_bits is None else wl.from_bits(gain_bits).cuda()
    r = torch.from_numpy(rms).cuda()
    esz = 4 if fp32_out else 2
    dfull, dbytes = gu.guarded(T * D * esz)
    dx = dbytes.view(torch.float32 if fp32_out else torch.bfloat16).view(T, D)
    gfull, gbytes = gu.guarded(D * 4)
    dgain = gbytes.view(torch.float32) if want_dgain else None
    wsb = binding.mxnorm_bwd_workspace_bytes(T, D)
    wfull, ws = gu.guarded(wsb)
    binding.mxnorm_bwd(x, g, gain, r, dx, dgain, ws if want_dgain else None)
    torch.cuda.synchronize()
    assert gu.guards_intact(dfull, T * D * esz) and gu.guards_intact(gfull, D * 4) and gu.guards_intact(wfull, wsb)
    dx_np = dx.float().cpu().numpy().astype(np.float64) if not fp32_out else dx.cpu().numpy().astype(np.float64)
    dx_bits = None if fp32_out else dx.cpu().view(torch.int16).numpy().view(np.uint16)
    return dx_np, dx_bits, (None if dgain is None else dgain.cpu().numpy().astype(np.float64))


def check(binding, oracle, T, D, seed, with_gain=True):
    w = wl.Workload("t", T, D, seed=seed, outlier_frac=0.002, has_gain=True, has_grad=True)
    inp = wl.make_inputs(w)
    x, g = wl.bits(inp["x"]), wl.bits(inp["grad"])
    gain = wl.bits(inp["gain"]) if with_gain else None
    if D % 32 == 0:
        _, _, rms = oracle.mxnorm_ref(x, eps=1e-5)            # the estimate the forward would save
    else:                                                     # any positive r is a valid input of the backward
        xv = (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        rms = (1.07 * np.sqrt((xv ** 2).mean(-1)) + 1e-5).astype(np.float32)
    want_dx, want_dg = oracle.mxnorm_bwd_ref(x, g, gain, rms)
    # fp32 output: per-row max-norm relative 1e-3 (binary32 row dot and products against binary64)
    dx, _, dg = run_bwd(binding, x, g, gain, rms, fp32_out=True)
    row_scale = np.abs(want_dx).max(-1, keepdims=True)
    assert np.all(np.abs(dx - want_dx) <= 1e-3 * row_scale), np.max(np.abs(dx - want_dx) / row_scale)
    assert np.max(np.abs(dx - want_dx) / row_scale) < 1e-5       # in practice ~1e-7
    assert np.all(np.abs(dg - want_dg) <= 1e-3 * np.abs(want_dg).max())
    # bf16 output: each element within one bf16 ulp of the correctly rounded oracle value
    dxb, bits, dg2 = run_bwd(binding, x, g, gain, rms, fp32_out=False)
    assert np.all(np.abs(dxb - want_dx) <= 1.0 * bf16_ulp(want_dx) + 1e-3 * 2.0 ** -8 * row_scale)
    assert np.array_equal(dg, dg2)
    # dX only (no workspace needed)
    dx3, _, none = run_bwd(binding, x, g, gain, rms, fp32_out=True, want_dgain=False)
    assert none is None and np.array_equal(dx3, dx)
    return dx, dg


@pytest.mark.parametrize("D", [1536, 2048, 3072])
def test_backward_with_many_rows(binding, oracle, D):
    """From 32768 rows on the launcher takes fewer CTAs per SM or a shallower ring for some row lengths: every row of dX
    and the gain gradient against the oracle, with and without the gain gradient (the two use different launch plans)."""
    T = 32768 + 3
    w = wl.Workload("t", T, D, seed=40 + D, outlier_frac=0.002, has_gain=True, has_grad=True)
    inp = wl.make_inputs(w)
    x, g, gain = wl.bits(inp["x"]), wl.bits(inp["grad"]), wl.bits(inp["gain"])
    _, _, rms = oracle.mxnorm_ref(x, eps=1e-5)
    want_dx, want_dg = oracle.mxnorm_bwd_ref(x, g, gain, rms)
    row_scale = np.abs(want_dx).max(-1, keepdims=True)
    dx, _, dg = run_bwd(binding, x, g, gain, rms, fp32_out=True)
    assert np.max(np.abs(dx - want_dx) / row_scale) < 1e-5
    assert np.all(np.abs(dg - want_dg) <= 1e-3 * np.abs(want_dg).max())
    dx2, _, none = run_bwd(binding, x, g, gain, rms, fp32_out=True, want_dgain=False)
    assert none is None and np.array_equal(dx2, dx)


@pytest.mark.parametrize("T,D", [(1, 8), (3, 64), (37, 768), (130, 1024), (65, 2048), (33, 4096), (7, 2056),
                                 (5, 8192), (4, 16384), (1000, 512), (900, 1024), (700, 2048), (9, 5120), (300, 5120), (7, 6144), (300, 8192), (500, 3072), (300, 7168), (450, 1536), (150, 10240), (150, 12288), (150, 14336), (150, 16384), (7, 8200), (5, 9000), (40, 12296)])
def test_backward_matches_oracle(binding, oracle, T, D):
    check(binding, oracle, T, D, seed=T + D)
    check(binding, oracle, T, D, seed=T + D + 1, with_gain=False)


def test_backward_is_repeatable_and_sums_all_rows(binding, oracle):
    a = check(binding, oracle, 1500, 1024, seed=5)
    b = check(binding, oracle, 1500, 1024, seed=5)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_backward_with_true_rms_is_orthogonal_to_x(binding, oracle):
    w = wl.Workload("t", 64, 2048, seed=9, has_gain=True, has_grad=True)
    inp = wl.make_inputs(w)
    x, g, gain = wl.bits(inp["x"]), wl.bits(inp["grad"]), wl.bits(inp["gain"])
    _, _, rms = oracle.rmsnorm_mxfp8_ref(x)
    dx, _, _ = run_bwd(binding, x, g, gain, rms, fp32_out=True)
    xv = (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    assert np.all(np.abs((dx * xv).sum(-1)) <= 1e-4 * np.abs(dx * xv).sum(-1))


def test_backward_with_zero_rows_matches_the_forward_convention(binding, oracle):
    """Rows of zeros (padding tokens) among normal rows: the forward saves r~ = 0 for them; the backward must give
    dX = 0 there and a finite dgamma that equals the oracle's (which adds nothing for those rows)."""
    w = wl.Workload("t", 700, 1024, seed=13, outlier_frac=0.002, has_gain=True, has_grad=True)
    inp = wl.make_inputs(w)
    x, g, gain = wl.bits(inp["x"]).copy(), wl.bits(inp["grad"]), wl.bits(inp["gain"])
    zero_rows = [0, 3, 295, 296, 699]
    x[zero_rows] = 0
    x[3, ::2] = 0x8000
    # the r~ the library's own forward saves
    xg = wl.from_bits(x).cuda()
    codes, scales, rms = binding.alloc_outputs(700, 1024)
    binding.mxnorm_fwd(xg, None, codes, scales, rms, eps=1e-5)
    torch.cuda.synchronize()
    r = rms.cpu().numpy()
    assert np.all(r[zero_rows] == 0) and np.array_equal(r, oracle.mxnorm_ref(x, eps=1e-5)[2])
    want_dx, want_dg = oracle.mxnorm_bwd_ref(x, g, gain, r)
    for fp32_out in (True, False):
        dx, _, dg = run_bwd(binding, x, g, gain, r, fp32_out=fp32_out)
        assert np.all(np.isfinite(dx)) and np.all(np.isfinite(dg))
        assert np.all(dx[zero_rows] == 0)
        scale = np.maximum(np.abs(want_dx).max(-1, keepdims=True), 1e-30)
        tol = 1e-3 if fp32_out else 2.0 ** -7
        assert np.all(np.abs(dx - want_dx) <= tol * scale)
        assert np.all(np.abs(dg - want_dg) <= 1e-3 * np.abs(want_dg).max())
    assert binding.device_timeouts() == 0


def test_a_bounded_wait_that_runs_out_is_counted_and_the_context_stays_usable(binding, oracle):
    """The only device-side waits of the library are the bounded mbarrier waits of the backward's copy ring.  A test
    kernel makes such a wait run out (a barrier nobody completes, a few thousand polls): the event must be counted,
    reported as MXN_ERR_TIMEOUT, resettable, and later launches must work as before."""
    assert binding.device_timeouts() == 0
    binding.selftest_bounded_wait(3000)
    n = ctypes.c_uint(0)
    st = binding.lib.mxn_device_timeouts(ctypes.byref(n))
    assert st == 7 and n.value == 1 and "wait" in binding.status_string(st)
    binding.selftest_bounded_wait(100)
    assert binding.device_timeouts() == 2
    binding.device_timeouts_reset()
    assert binding.device_timeouts() == 0
    assert binding.lib.mxn_selftest_bounded_wait(0, None) == 2 and binding.lib.mxn_selftest_bounded_wait(1 << 20, None) == 2
    check(binding, oracle, 65, 2048, seed=3)          # the context is intact: a full backward still matches the oracle
    assert binding.device_timeouts() == 0
