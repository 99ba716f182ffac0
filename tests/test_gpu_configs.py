"""GPU parity on the five benchmark configurations at full size, in the launch configuration the
benchmark times.  The C oracle is fast enough to compare every element."""
import numpy as np
import pytest
import torch

from paper_2603_13180_b200 import workloads as wl
from tests import gpu_util as gu
from tests.test_gpu_backward import run_bwd

pytestmark = pytest.mark.gpu

EPS = 1e-5


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_13180_b200 import binding as b
    return b


@pytest.mark.parametrize("name", ["C1", "C2", "C3"])
def test_mxfp8_configs_full_size(binding, oracle, name):
    w = wl.CONFIGS[name]
    inp = wl.make_inputs(w)
    x = wl.bits(inp["x"])
    gain = None if inp["gain"] is None else wl.bits(inp["gain"])
    layout = 1 if w.swizzled_scales else 0
    # the method (gain folded into the next weight) - bit exact
    got = gu.run_fwd(binding, oracle, "mx", x, eps=EPS, layout=layout)
    gu.assert_exact(got, gu.run_ref(oracle, "mx", x, eps=EPS), f"{name} mxnorm_fwd")
    # plain cast - bit exact
    got = gu.run_fwd(binding, oracle, "cast", x, layout=layout)
    gu.assert_exact(got, gu.run_ref(oracle, "cast", x), f"{name} mx_cast")
    # the conventional baseline, without and with its gain - within the rounding of rho
    for g in (None, gain):
        got = gu.run_fwd(binding, oracle, "rms", x, g, eps=EPS, layout=layout)
        flipped, stepped = gu.assert_within_rounding_of_rho(got, gu.run_ref(oracle, "rms", x, g, eps=EPS), 32,
                                                            f"{name} rmsnorm_mxfp8_fwd")
        print(f"{name} rmsnorm gain={g is not None}: {flipped} scale bytes and {stepped} codes differ by one step")
    if gain is not None:
        got = gu.run_fwd(binding, oracle, "mx", x, gain, eps=EPS, layout=layout)
        gu.assert_exact(got, gu.run_ref(oracle, "mx", x, gain, eps=EPS), f"{name} mxnorm_fwd with gain")


@pytest.mark.parametrize("block", [16, 64])
def test_other_block_sizes_at_the_benchmark_shape(binding, oracle, block):
    """[16384, 4096] with blocks of 16 and 64 (two lanes share a block of 64), E4M3 and E2M1 codes, tiled scales."""
    x = wl.bits(wl.make_inputs(wl.CONFIGS["C3"])["x"])
    got = gu.run_fwd(binding, oracle, "mx", x, block=block, eps=EPS, layout=1)
    gu.assert_exact(got, gu.run_ref(oracle, "mx", x, block=block, eps=EPS), f"mxnorm_fwd B={block}")
    got = gu.run_fwd(binding, oracle, "mx4", x, block=block, eps=EPS, layout=1)
    gu.assert_exact(got, gu.run_ref(oracle, "mx4", x, block=block, eps=EPS), f"mxnorm_mxfp4_fwd B={block}")


def test_nvfp4_config_full_size(binding, oracle):
    w = wl.CONFIGS["C4"]
    x = wl.bits(wl.make_inputs(w)["x"])
    got = gu.run_fwd(binding, oracle, "nvfp4", x, eps=EPS)
    gu.assert_exact(got, gu.run_ref(oracle, "nvfp4", x, eps=EPS), "C4 mxnorm_nvfp4_fwd")


def test_backward_config_full_size(binding, oracle):
    w = wl.CONFIGS["C5"]
    inp = wl.make_inputs(w)
    x, g, gain = wl.bits(inp["x"]), wl.bits(inp["grad"]), wl.bits(inp["gain"])
    _, _, rms = oracle.mxnorm_ref(x, eps=EPS)
    # dgamma over all 16384 rows (the oracle's column sum is a serial loop) and every row of dX (rows in parallel),
    # compared chunk by chunk to bound the host memory of the binary64 reference
    dx, _, dg = run_bwd(binding, x, g, gain, rms, fp32_out=True)
    _, want_dg = oracle.mxnorm_bwd_ref(x, g, gain, rms, want_dx=False)
    assert np.all(np.abs(dg - want_dg) <= 1e-3 * np.abs(want_dg).max())
    dxb, _, dg2 = run_bwd(binding, x, g, gain, rms, fp32_out=False)
    assert np.array_equal(dg, dg2)
    worst = 0.0
    for r0 in range(0, w.T, 2048):
        sel = slice(r0, r0 + 2048)
        want_dx, _ = oracle.mxnorm_bwd_ref(x[sel], g[sel], gain, rms[sel], want_dgain=False)
        scale = np.abs(want_dx).max(-1, keepdims=True)
        err = np.abs(dx[sel] - want_dx)
        assert np.all(err <= 1e-3 * scale)
        worst = max(worst, float((err / scale).max()))
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want_dx), 2.0 ** -126))) - 7)
        assert np.all(np.abs(dxb[sel] - want_dx) <= ulp + 1e-3 * 2.0 ** -8 * scale)
    assert worst < 1e-5          # in practice ~2e-7 of the row maximum
