"""Sizes beyond 2^31 elements: index arithmetic must be 64-bit everywhere.  Inputs are generated on the GPU (seeded) and
sampled rows are checked against the oracle."""
import numpy as np
import pytest
import torch

from paper_2603_13180_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_13180_b200 import binding as b
    return b


def _big_input(T, D, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    x = torch.empty((T, D), dtype=torch.bfloat16, device="cuda")
    step = 65536
    for t in range(0, T, step):
        n = min(step, T - t)
        x[t:t + n] = (torch.randn(n, D, generator=g, device="cuda") * torch.exp(torch.randn(n, 1, generator=g, device="cuda"))).to(torch.bfloat16)
    return x


def test_forward_and_backward_beyond_2_31_elements(binding, oracle):
    T, D = 540_001, 4096                         # 2.21e9 elements; odd T: ragged last CTA and last scale tile
    x = _big_input(T, D, seed=7)
    layout = binding.SCALES_SWIZZLE_128x4
    codes, scales, rms = binding.alloc_outputs(T, D, 32, layout)
    binding.mxnorm_fwd(x, None, codes, scales, rms, eps=1e-5, layout=layout)
    torch.cuda.synchronize()
    sel = np.unique(np.concatenate([np.arange(0, T, 40009), [T - 1, T - 2, 524287, 524288, 524289]]))
    sel_t = torch.from_numpy(sel).cuda()
    xs = wl.bits(x[sel_t].cpu())
    wc, ws, wr = oracle.mxnorm_ref(xs, eps=1e-5)
    assert np.array_equal(codes[sel_t].cpu().numpy(), wc)
    assert np.array_equal(rms[sel_t].cpu().numpy(), wr)
    K = D // 32
    offs = torch.from_numpy(oracle.swizzle_index_map(T, K)[sel]).cuda()        # byte offsets of the sampled rows' scales
    assert np.array_equal(scales[offs].cpu().numpy(), ws)
    # backward on the same tensor (dX only; x doubles as the upstream gradient)
    dx = torch.empty_like(x)
    binding.mxnorm_bwd(x, x, None, rms, dx, None, None)
    torch.cuda.synchronize()
    want_dx, _ = oracle.mxnorm_bwd_ref(xs, xs, None, wr, want_dgain=False)
    got = dx[sel_t].float().cpu().numpy().astype(np.float64)
    scale = np.abs(want_dx).max(-1, keepdims=True)
    assert np.all(np.abs(got - want_dx) <= 2.0 ** -8 * scale + 2.0 ** -8 * np.abs(want_dx))
    del dx, codes, scales
    # column-wise cast: T must be a multiple of 32
    T2 = 540_000 - 540_000 % 32
    ct = torch.empty((D, T2), dtype=torch.uint8, device="cuda")
    st = torch.empty((D * (T2 // 32),), dtype=torch.uint8, device="cuda")
    binding.mx_cast_transposed(x[:T2], rms[:T2].contiguous(), ct, st, eps=1e-5)
    torch.cuda.synchronize()
    cols = [0, 1, 2047, 4095]
    for t0 in (0, 262144 - 32, 524288, T2 - 32):          # token blocks on both sides of element index 2^31
        blk = wl.bits(x[t0:t0 + 32].cpu())
        wct, wst = oracle.mx_cast_transposed_ref(blk, rms=rms[t0:t0 + 32].cpu().numpy(), eps=1e-5)
        assert np.array_equal(ct[cols, t0:t0 + 32].cpu().numpy(), wct[cols])
        assert np.array_equal(st.view(D, T2 // 32)[cols, t0 // 32].cpu().numpy(), wst[cols, 0])


def test_token_counts_beyond_65535_tiles(binding, oracle):
    """Very long, narrow tensors: more than 65535 token tiles in the column-wise cast and more than 2^21 rows in the
    row-wise kernels (grids are one-dimensional, so only the total number of CTAs is bounded)."""
    T, D = 65537 * 32, 64                        # 2,097,184 tokens
    x = _big_input(T, D, seed=9)
    codes, scales, rms = binding.alloc_outputs(T, D, 32, binding.SCALES_ROWMAJOR)
    binding.mxnorm_fwd(x, None, codes, scales, rms, eps=1e-5)
    ct = torch.empty((D, T), dtype=torch.uint8, device="cuda")
    st = torch.empty((D, T // 32), dtype=torch.uint8, device="cuda")
    binding.mx_cast_transposed(x, rms, ct, st, eps=1e-5)
    torch.cuda.synchronize()
    xb = wl.bits(x.cpu())
    wc, ws, wr = oracle.mxnorm_ref(xb, eps=1e-5)
    assert np.array_equal(codes.cpu().numpy(), wc)
    assert np.array_equal(scales.cpu().numpy().reshape(T, D // 32), ws)
    assert np.array_equal(rms.cpu().numpy(), wr)
    wct, wst = oracle.mx_cast_transposed_ref(xb, rms=wr, eps=1e-5)
    assert np.array_equal(ct.cpu().numpy(), wct)
    assert np.array_equal(st.cpu().numpy(), wst)
