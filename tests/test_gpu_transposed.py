"""GPU parity of mx_cast_transposed (column-wise MXCast for the weight-gradient GEMM) against the oracle."""
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


def run(binding, oracle, x_bits, rms, eps=0.0, round=0, layout=0):
    T, D = x_bits.shape
    x = wl.from_bits(x_bits).cuda()
    r = None if rms is None else torch.from_numpy(np.ascontiguousarray(rms, dtype=np.float32)).cuda()
    cfull, codes = gu.guarded(D * T)
    sbytes = binding.scale_bytes(D, T // 32, layout)
    sfull, scales = gu.guarded(sbytes)
    codes.fill_(0x5A)
    scales.fill_(0x5A)
    binding.mx_cast_transposed(x, r, codes, scales, eps=eps, round=round, layout=layout)
    torch.cuda.synchronize()
    assert gu.guards_intact(cfull, D * T) and gu.guards_intact(sfull, sbytes)
    s_np = scales.cpu().numpy()
    if layout == 1:
        assert gu.swizzle_padding_is_zero(s_np, D, T // 32, oracle)
        s_np = gu.unswizzle(s_np, D, T // 32, oracle)
    else:
        s_np = s_np.reshape(D, T // 32)
    return codes.cpu().numpy().reshape(D, T), s_np


@pytest.mark.parametrize("T,D", [(32, 4), (64, 128), (96, 160), (160, 132), (256, 4096), (2048, 768), (128, 5120),
                                 (32, 64), (288, 72), (416, 200), (1024, 1280)])
def test_transposed_cast_matches_oracle_bit_for_bit(binding, oracle, T, D):
    inp = wl.make_inputs(wl.Workload("t", T, D, seed=T + D, outlier_frac=0.01 if D >= 100 else 0.0))
    x = wl.bits(inp["x"])
    xv = (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    r_est = (0.97 * np.sqrt((xv ** 2).mean(-1))).astype(np.float32)      # any positive r is a valid normaliser
    for rms, eps in ((None, 0.0), (r_est, 1e-5), (r_est, 0.0)):
        c, s = run(binding, oracle, x, rms, eps=eps)
        wc, ws = oracle.mx_cast_transposed_ref(x, rms=rms, eps=eps)
        assert np.array_equal(s, ws), f"{np.count_nonzero(s != ws)} scales differ"
        assert np.array_equal(c, wc), f"{np.count_nonzero(c != wc)} codes differ"
    for rnd in (1, 2):
        c, s = run(binding, oracle, x, r_est, eps=1e-5, round=rnd)
        wc, ws = oracle.mx_cast_transposed_ref(x, rms=r_est, eps=1e-5, mode=rnd)
        assert np.array_equal(s, ws) and np.array_equal(c, wc)
    c, s = run(binding, oracle, x, r_est, eps=1e-5, layout=1)
    wc, ws = oracle.mx_cast_transposed_ref(x, rms=r_est, eps=1e-5)
    assert np.array_equal(s, ws) and np.array_equal(c, wc)


def test_transposed_cast_full_size_with_the_forward_estimate(binding, oracle):
    """Config C5's tensors: X [16384, 4096] and the r~ that mxnorm_fwd saves; zero and tiny rows included."""
    inp = wl.make_inputs(wl.CONFIGS["C5"])
    x = wl.bits(inp["x"]).copy()
    x[5] = 0
    x[77] = 0x0080
    _, _, r_est = oracle.mxnorm_ref(x, eps=1e-5)
    c, s = run(binding, oracle, x, r_est, eps=1e-5, layout=1)
    wc, ws = oracle.mx_cast_transposed_ref(x, rms=r_est, eps=1e-5)
    assert np.array_equal(s, ws) and np.array_equal(c, wc)
    g = wl.bits(inp["grad"])
    c, s = run(binding, oracle, g, None)
    wc, ws = oracle.mx_cast_transposed_ref(g)
    assert np.array_equal(s, ws) and np.array_equal(c, wc)


def test_transposed_cast_of_an_input_that_is_only_8_byte_aligned(binding, oracle):
    """A contiguous view whose base address is 8 mod 16 is valid input (the contract asks for 8 bytes): it must take
    the register kernel with 8-byte loads, not the kernel that stages rows with 16-byte copies."""
    T, D = 160, 256
    inp = wl.make_inputs(wl.Workload("t", T, D, seed=77, outlier_frac=0.01))
    x_bits = wl.bits(inp["x"])
    buf = torch.zeros(T * D + 4, dtype=torch.bfloat16, device="cuda")
    assert buf.data_ptr() % 16 == 0
    x = buf[4:].view(T, D)                                   # base address = 8 mod 16
    x.copy_(inp["x"])
    assert x.data_ptr() % 16 == 8 and x.is_contiguous()
    xv = (x_bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    r_est = (1.03 * np.sqrt((xv ** 2).mean(-1))).astype(np.float32)
    r = torch.from_numpy(r_est).cuda()
    for layout in (0, 1):
        cfull, codes = gu.guarded(D * T)
        sbytes = binding.scale_bytes(D, T // 32, layout)
        sfull, scales = gu.guarded(sbytes)
        binding.mx_cast_transposed(x, r, codes, scales, eps=1e-5, layout=layout)
        torch.cuda.synchronize()
        assert gu.guards_intact(cfull, D * T) and gu.guards_intact(sfull, sbytes)
        wc, ws = oracle.mx_cast_transposed_ref(x_bits, rms=r_est, eps=1e-5)
        s_np = scales.cpu().numpy()
        s_np = gu.unswizzle(s_np, D, T // 32, oracle) if layout == 1 else s_np.reshape(D, T // 32)
        assert np.array_equal(s_np, ws) and np.array_equal(codes.cpu().numpy().reshape(D, T), wc)
    # the E5M2 variant shares the dispatch
    cfull, codes = gu.guarded(D * T)
    sfull, scales = gu.guarded(D * (T // 32))
    binding.mx_cast_transposed_e5m2(x, codes, scales)
    torch.cuda.synchronize()
    wc, ws = oracle.mx_cast_transposed_ref(x_bits, elem=oracle.ELEM_E5M2)
    assert np.array_equal(scales.cpu().numpy().reshape(D, T // 32), ws) and np.array_equal(codes.cpu().numpy().reshape(D, T), wc)


def test_transposed_cast_argument_errors(binding):
    L = binding.lib
    fake = 0x7F0000000000
    assert L.mx_cast_transposed(fake, None, 100, 128, 0.0, fake, fake, 0, 0, None) == 2     # T % 32
    assert L.mx_cast_transposed(fake, None, 128, 130, 0.0, fake, fake, 0, 0, None) == 2     # D % 4
    assert L.mx_cast_transposed(fake, None, 0, 128, 0.0, fake, fake, 0, 0, None) == 0
    assert L.mx_cast_transposed(None, None, 128, 128, 0.0, fake, fake, 0, 0, None) == 1
    assert L.mx_cast_transposed(fake + 4, None, 128, 128, 0.0, fake, fake, 0, 0, None) == 3
    assert L.mx_cast_transposed(fake, None, 128, 128, 0.0, fake, fake, 5, 0, None) == 4


@pytest.mark.parametrize("T,D", [(64, 128), (96, 160), (256, 4096), (160, 132)])
def test_e5m2_casts_match_oracle_bit_for_bit(binding, oracle, T, D):
    """E5M2 codes (gradient tensors): row-wise and column-wise casts."""
    inp = wl.make_inputs(wl.Workload("t", T, D, seed=3 * T + D, outlier_frac=0.01, has_grad=True))
    g = wl.bits(inp["grad"])
    x = wl.from_bits(g).cuda()
    # column-wise
    cfull, codes = gu.guarded(D * T)
    sfull, scales = gu.guarded(binding.scale_bytes(D, T // 32, 0))
    binding.mx_cast_transposed_e5m2(x, codes, scales)
    torch.cuda.synchronize()
    assert gu.guards_intact(cfull, D * T) and gu.guards_intact(sfull, D * (T // 32))
    wc, ws = oracle.mx_cast_transposed_ref(g, elem=oracle.ELEM_E5M2)
    assert np.array_equal(scales.cpu().numpy().reshape(D, T // 32), ws)
    assert np.array_equal(codes.cpu().numpy().reshape(D, T), wc)
    # row-wise, all block sizes that divide D
    for B in (16, 32, 64):
        if D % B:
            continue
        cfull, codes = gu.guarded(T * D)
        sfull, scales = gu.guarded(T * (D // B))
        binding.mx_cast_e5m2(x, codes, scales, block=B)
        torch.cuda.synchronize()
        assert gu.guards_intact(cfull, T * D) and gu.guards_intact(sfull, T * (D // B))
        wc, ws = oracle.mx_cast_ref(g, block=B, elem=oracle.ELEM_E5M2)
        assert np.array_equal(scales.cpu().numpy().reshape(T, D // B), ws)
        assert np.array_equal(codes.cpu().numpy().reshape(T, D), wc)


def test_e5m2_all_bf16_patterns(binding, oracle):
    pats = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    pats = pats[(pats & 0x7F80) != 0x7F80]
    xb = np.zeros((pats.size, 32), np.uint16)
    xb[:, 0] = pats
    xb[:, 9] = (pats >> 1) & 0x7FFF
    xb[(xb[:, 9] & 0x7F80) == 0x7F80, 9] = 0
    x = wl.from_bits(xb).cuda()
    codes = torch.empty((pats.size, 32), dtype=torch.uint8, device="cuda")
    scales = torch.empty((pats.size,), dtype=torch.uint8, device="cuda")
    binding.mx_cast_e5m2(x, codes, scales)
    torch.cuda.synchronize()
    wc, ws = oracle.mx_cast_ref(xb, elem=oracle.ELEM_E5M2)
    assert np.array_equal(scales.cpu().numpy().reshape(-1, 1), ws) and np.array_equal(codes.cpu().numpy(), wc)
