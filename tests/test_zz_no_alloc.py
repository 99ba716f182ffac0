"""mxnorm_bwd_noalloc: the backward for callers that cannot allocate a workspace (ops inside a fixed
memory plan, plug-ins that only see the op's tensors).  Its dgain partial sums live in an 8 MiB array
built into the library, shared by every call on the device.  This file is collected last on purpose:
if the built-in scratch misbehaves, every other test has already run.

The GPU test calls the new entry point through the C ABI twice in a row, on different inputs, and
checks each result against the existing mxnorm_bwd (caller-provided workspace): within the tolerance the
backward tests use, and - because both entry points launch the same kernels on the same inputs - bit for bit;
the second call has fewer partial rows than the first, so stale scratch contents
from the first call would show up in its dgain."""
import numpy as np
import pytest
import torch

from paper_2603_13180_b200 import workloads as wl

ROW_TOL = 1e-3   # per-row max-norm tolerance of the backward tests


def _inputs(T, D, seed):
    w = wl.Workload("t", T, D, seed=seed, outlier_frac=0.002, has_gain=True, has_grad=True)
    inp = wl.make_inputs(w)
    x = inp["x"].cuda()
    g = inp["grad"].cuda()
    gain = inp["gain"].cuda()
    rms = (1.05 * x.float().pow(2).mean(-1).sqrt() + 1e-5).contiguous()   # any positive r is a valid input
    return x, g, gain, rms


def _both(mx, T, D, seed, out_dtype):
    x, g, gain, rms = _inputs(T, D, seed)
    dx_a = torch.empty((T, D), dtype=out_dtype, device="cuda")
    dg_a = torch.empty((D,), dtype=torch.float32, device="cuda")
    ws = torch.empty(mx.mxnorm_bwd_workspace_bytes(T, D), dtype=torch.uint8, device="cuda")
    mx.mxnorm_bwd(x, g, gain, rms, dx_a, dg_a, ws)
    dx_b = torch.full((T, D), float("nan"), dtype=out_dtype, device="cuda")
    dg_b = torch.full((D,), float("nan"), dtype=torch.float32, device="cuda")
    mx.mxnorm_bwd_noalloc(x, g, gain, rms, dx_b, dg_b)
    torch.cuda.synchronize()
    return dx_a.float().cpu().numpy(), dg_a.cpu().numpy(), dx_b.float().cpu().numpy(), dg_b.cpu().numpy()


def _close(dx_a, dg_a, dx_b, dg_b):
    scale = np.abs(dx_a).max(-1, keepdims=True)
    assert np.all(np.isfinite(dx_b)) and np.all(np.isfinite(dg_b))
    assert np.all(np.abs(dx_b - dx_a) <= ROW_TOL * scale)
    assert np.all(np.abs(dg_b - dg_a) <= ROW_TOL * np.abs(dg_a).max())
    assert np.array_equal(dx_a, dx_b) and np.array_equal(dg_a, dg_b)     # same kernels, same inputs: identical bits


@pytest.mark.gpu
def test_noalloc_backward_matches_workspace_backward_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_13180_b200 import binding as mx
    assert mx.lib.mxnorm_bwd_noalloc_max_scratch_bytes() == 8 << 20
    # first call: 296 partial rows of 4096 floats (4.6 MiB of the 8 MiB); second: 100 partial rows, other data
    _close(*_both(mx, 1200, 4096, seed=1, out_dtype=torch.float32))
    _close(*_both(mx, 100, 4096, seed=2, out_dtype=torch.bfloat16))
    # and once more with the first shape, after the smaller call
    _close(*_both(mx, 1200, 4096, seed=3, out_dtype=torch.bfloat16))
    # dX alone uses no scratch at all: any supported size goes through
    x, g, gain, rms = _inputs(300, 16384, seed=4)
    dx = torch.empty((300, 16384), dtype=torch.float32, device="cuda")
    mx.mxnorm_bwd_noalloc(x, g, gain, rms, dx, None)
    dx_ref = torch.empty_like(dx)
    mx.mxnorm_bwd(x, g, gain, rms, dx_ref, None, None)
    torch.cuda.synchronize()
    assert torch.equal(dx, dx_ref)


def test_noalloc_backward_rejects_what_does_not_fit():
    """Needs no GPU: the size check comes before anything touches the device."""
    from paper_2603_13180_b200 import build
    build.build_library()
    from paper_2603_13180_b200 import binding as mx
    fake = 0x7F0000000000
    cap = mx.lib.mxnorm_bwd_noalloc_max_scratch_bytes()
    assert mx.mxnorm_bwd_workspace_bytes(4096, 16384) > cap
    st = mx.lib.mxnorm_bwd_noalloc(fake, fake, None, fake, 4096, 16384, fake, 0, fake, None)
    assert st == 8 and "scratch" in mx.status_string(st)
    assert mx.lib.mxnorm_bwd_noalloc(fake, fake, None, fake, 64, 4100, fake, 0, fake, None) == 2
    assert mx.lib.mxnorm_bwd_noalloc(None, fake, None, fake, 64, 4096, fake, 0, fake, None) == 1
    assert mx.lib.mxnorm_bwd_noalloc(fake + 2, fake, None, fake, 64, 4096, fake, 0, fake, None) == 3
