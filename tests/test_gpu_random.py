"""Randomised differential test: seeded random shapes, block sizes, layouts, statistics and value mixes
(zeros, negative zeros, subnormals, huge and tiny magnitudes, whole zero rows and blocks) through every
bit-exact forward entry point, compared byte for byte with the CPU oracle."""
import numpy as np
import pytest
import torch

from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_13180_b200 import binding as b
    return b


def f32_to_bf16_bits(v: np.ndarray) -> np.ndarray:
    """round-to-nearest-even truncation of binary32 to bf16 bit patterns (finite inputs)"""
    u = v.astype(np.float32).view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


def random_rows(rng: np.random.Generator, T: int, D: int, block: int) -> np.ndarray:
    """bf16 bit patterns [T, D]: Gaussian rows with a log-uniform row scale inside the tested domain, plus special values"""
    scale = 2.0 ** rng.uniform(-30, 30, size=(T, 1))
    x = rng.standard_normal((T, D)) * scale
    kind = rng.integers(0, 6)
    if kind == 1:                                   # heavy tails
        x *= np.exp(2.0 * rng.standard_normal((T, D)))
    elif kind == 2:                                 # sparse: most elements exactly zero
        x *= rng.random((T, D)) < 0.05
    elif kind == 3:                                 # whole zero blocks and a whole zero row
        nb = D // block
        x = x.reshape(T, nb, block) * (rng.random((T, nb, 1)) < 0.7)
        x = x.reshape(T, D)
        x[rng.integers(0, T)] = 0.0
    elif kind == 4:                                 # exact powers of two and ties of the element format
        x = np.ldexp(rng.choice([1.0, 1.0625, 1.125, 1.25, 1.5, 1.75, 1.875], size=(T, D)), rng.integers(-8, 9, size=(T, D)))
        x *= rng.choice([-1.0, 1.0], size=(T, D))
    bits = f32_to_bf16_bits(np.clip(x, -3e38, 3e38))
    # sprinkle negative zeros and bf16 subnormals
    m = rng.random((T, D))
    bits = np.where(m < 0.002, np.uint16(0x8000), bits)
    bits = np.where((m >= 0.002) & (m < 0.004), rng.integers(1, 0x80, size=(T, D)).astype(np.uint16), bits)
    bits = bits.astype(np.uint16)
    # a row without a single normal value has an RMS outside the binary32 normal range (outside the stated domain):
    # make such rows exactly zero (signs kept)
    normal = ((bits >> 7) & 0xFF) != 0
    bits = np.where(normal.any(axis=1, keepdims=True), bits, bits & np.uint16(0x8000))
    return np.ascontiguousarray(bits)


def pick_shape(rng, block):
    T = int(rng.choice([1, 2, 3, 5, 17, 64, 127, 129, 200, 333]))
    k = int(rng.choice([1, 2, 3, 7, 24, 31, 32, 33, 40, 63, 64, 65, 96, 100, 128, 160, 192, 224, 250, 256, 320, 384, 512]))
    D = k * block
    while D > 32768:
        D //= 2
    D -= D % block
    return T, max(D, block)


@pytest.mark.parametrize("seed", range(40))
def test_random_cases_match_the_oracle_bit_for_bit(binding, oracle, seed):
    rng = np.random.default_rng(1000 + seed)
    for _ in range(4):
        block = int(rng.choice([16, 32, 64]))
        T, D = pick_shape(rng, block)
        x = random_rows(rng, T, D, block)
        layout = int(rng.integers(0, 2))
        eps = float(rng.choice([0.0, 1e-5, 1e-2]))
        p = int(rng.choice([1, 2]))
        what = f"seed {seed}: T={T} D={D} B={block} layout={layout} eps={eps} p={p}"
        got = gu.run_fwd(binding, oracle, "mx", x, block=block, p=p, eps=eps, layout=layout)
        gu.assert_exact(got, gu.run_ref(oracle, "mx", x, block=block, p=p, eps=eps), "mxnorm_fwd " + what)
        rnd = int(rng.integers(0, 3))
        got = gu.run_fwd(binding, oracle, "cast", x, block=block, round=rnd, layout=layout)
        gu.assert_exact(got, gu.run_ref(oracle, "cast", x, block=block, round=rnd), f"mx_cast round={rnd} " + what)
        got = gu.run_fwd(binding, oracle, "mx4", x, block=block, p=p, eps=eps, layout=layout)
        gu.assert_exact(got, gu.run_ref(oracle, "mx4", x, block=block, p=p, eps=eps), "mxnorm_mxfp4_fwd " + what)
        got = gu.run_fwd(binding, oracle, "cast4", x, block=block, layout=layout)
        gu.assert_exact(got, gu.run_ref(oracle, "cast4", x, block=block), "mx_cast_fp4 " + what)
        # gain vector: magnitudes over twenty binades, both signs, some exact zeros
        g = rng.standard_normal(D) * 2.0 ** rng.uniform(-10, 10, size=D) * (rng.random(D) > 0.02)
        gain = f32_to_bf16_bits(g)
        got = gu.run_fwd(binding, oracle, "mx", x, gain, block=block, p=p, eps=eps, round=rnd, layout=layout)
        gu.assert_exact(got, gu.run_ref(oracle, "mx", x, gain, block=block, p=p, eps=eps, round=rnd), f"mxnorm_fwd with gain round={rnd} " + what)
        if D % 16 == 0:
            got = gu.run_fwd(binding, oracle, "nvfp4", x, p=p, eps=eps, layout=layout)
            gu.assert_exact(got, gu.run_ref(oracle, "nvfp4", x, p=p, eps=eps), "mxnorm_nvfp4_fwd " + what)


@pytest.mark.parametrize("seed", range(12))
def test_random_training_side_cases(binding, oracle, seed):
    """The forward estimate feeding the column-wise cast, and the fused residual add, on the same random value mixes."""
    from paper_2603_13180_b200 import workloads as wl
    from tests.test_gpu_transposed import run as run_transposed
    rng = np.random.default_rng(5000 + seed)
    for _ in range(3):
        T = 32 * int(rng.choice([1, 2, 3, 5, 8]))
        D = int(rng.choice([8, 32, 96, 160, 264, 1024, 2048, 4096]))
        x = random_rows(rng, T, D, 8)
        xv = (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        r = np.sqrt((xv ** 2).mean(-1)).astype(np.float32)
        r[r == 0] = 1.0
        layout = int(rng.integers(0, 2))
        c, s = run_transposed(binding, oracle, x, r, eps=1e-5, layout=layout)
        wc, ws = oracle.mx_cast_transposed_ref(x, rms=r, eps=1e-5)
        assert np.array_equal(s, ws) and np.array_equal(c, wc), f"mx_cast_transposed seed {seed} T={T} D={D} layout={layout}"
    for _ in range(3):
        block = int(rng.choice([16, 32, 64]))
        T, D = pick_shape(rng, block)
        x, res = random_rows(rng, T, D, block), random_rows(rng, T, D, block)
        want_h, wc, ws, wr = oracle.mxnorm_add_ref(x, res, eps=1e-5, block=block)
        if not np.all(np.isfinite((want_h.astype(np.uint32) << 16).view(np.float32))):
            continue                                    # the sum overflowed bf16: outside the contract (finite inputs to the norm)
        xg, rg = wl.from_bits(x).cuda(), wl.from_bits(res).cuda()
        codes, scales, rms = binding.alloc_outputs(T, D, block)
        binding.mxnorm_add_fwd(xg, rg, xg, codes, scales, rms, eps=1e-5, block=block)      # in place
        torch.cuda.synchronize()
        what = f"mxnorm_add_fwd seed {seed} T={T} D={D} B={block}"
        assert np.array_equal(wl.bits(xg.cpu()), want_h), what
        assert np.array_equal(codes.cpu().numpy(), wc), what
        assert np.array_equal(scales.cpu().numpy().reshape(T, D // block), ws), what
        assert np.array_equal(rms.cpu().numpy(), wr), what
