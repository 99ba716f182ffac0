"""The entry points under CUDA stream capture: one training-step slice (forward, column-wise cast of the
saved activation, backward) captured once into a CUDA graph and replayed on fresh inputs must give the
same bytes as direct launches, and those match the CPU oracle."""
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


def _alloc(binding, T, D, layout):
    dev = "cuda"
    return {
        "x": torch.empty((T, D), dtype=torch.bfloat16, device=dev),
        "g": torch.empty((T, D), dtype=torch.bfloat16, device=dev),
        "codes": torch.empty((T, D), dtype=torch.uint8, device=dev),
        "scales": torch.zeros(binding.scale_bytes(T, D // 32, layout), dtype=torch.uint8, device=dev),
        "rms": torch.empty(T, dtype=torch.float32, device=dev),
        "codes_t": torch.empty((D, T), dtype=torch.uint8, device=dev),
        "scales_t": torch.zeros(binding.scale_bytes(D, T // 32, layout), dtype=torch.uint8, device=dev),
        "dx": torch.empty((T, D), dtype=torch.bfloat16, device=dev),
        "dgain": torch.empty(D, dtype=torch.float32, device=dev),
        "ws": torch.empty(binding.mxnorm_bwd_workspace_bytes(T, D), dtype=torch.uint8, device=dev),
    }


def _step(binding, b, gain, layout, eps):
    binding.mxnorm_fwd(b["x"], None, b["codes"], b["scales"], b["rms"], eps=eps, layout=layout)
    binding.mx_cast_transposed(b["x"], b["rms"], b["codes_t"], b["scales_t"], eps=eps, layout=layout)
    binding.mxnorm_bwd(b["x"], b["g"], gain, b["rms"], b["dx"], b["dgain"], b["ws"])


OUTPUTS = ("codes", "scales", "rms", "codes_t", "scales_t", "dx", "dgain")


@pytest.mark.parametrize("layout", [0, 1])
def test_captured_step_replays_bit_exactly(binding, oracle, layout):
    T, D, eps = 1504, 2048, 1e-5          # T: several CTAs per SM wave and a multiple of 32 for the column-wise cast
    w = wl.Workload("graph", T, D, seed=11, outlier_frac=0.002, has_gain=True, has_grad=True)
    first = wl.make_inputs(w)
    second = wl.make_inputs(wl.Workload("graph", T, D, seed=12, outlier_frac=0.002, has_gain=True, has_grad=True))
    gain = first["gain"].cuda()
    cap, ref = _alloc(binding, T, D, layout), _alloc(binding, T, D, layout)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        cap["x"].copy_(first["x"]); cap["g"].copy_(first["grad"])
        _step(binding, cap, gain, layout, eps)           # warm-up outside capture (first-call set-up happens here)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()

    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        _step(binding, cap, gain, layout, eps)

    for inp in (second, first, second):
        for k in OUTPUTS:                                 # every output byte, tile padding included, is rewritten
            cap[k].view(torch.uint8).fill_(0x5A)
            ref[k].view(torch.uint8).fill_(0xA5)
        cap["x"].copy_(inp["x"]); cap["g"].copy_(inp["grad"])
        graph.replay()
        ref["x"].copy_(inp["x"]); ref["g"].copy_(inp["grad"])
        _step(binding, ref, gain, layout, eps)
        torch.cuda.synchronize()
        assert binding.device_timeouts() == 0
        for k in OUTPUTS:
            a, b = cap[k].view(torch.uint8), ref[k].view(torch.uint8)
            assert torch.equal(a, b), f"{k}: graph replay differs from direct launches"

    # and the replayed bytes are the oracle's (last replay: `second`)
    xb = wl.bits(second["x"])
    want_codes, want_scales, want_rms = oracle.mxnorm_ref(xb, eps=eps)
    assert np.array_equal(cap["codes"].cpu().numpy(), want_codes)
    assert np.array_equal(cap["rms"].cpu().numpy(), want_rms)
    if layout == 0:
        assert np.array_equal(cap["scales"].cpu().numpy().reshape(T, D // 32), want_scales)
    tc, ts = oracle.mx_cast_transposed_ref(xb, want_rms, eps=eps)
    assert np.array_equal(cap["codes_t"].cpu().numpy(), tc)
    if layout == 0:
        assert np.array_equal(cap["scales_t"].cpu().numpy().reshape(D, T // 32), ts)


def test_consumer_kernel_right_behind_its_producer(binding, oracle):
    """Kernels ask for their input rows in L2 before they wait for the previous kernel of the stream.  When that previous
    kernel is the PRODUCER of those rows the early request may only ever be a hint: here mxnorm_add_fwd writes h and
    mxnorm_fwd reads h right behind it, at full size and with fresh data every iteration, and the consumer's bytes must be
    those of the producer's own fused MXNorm of h (and the oracle's on sampled rows)."""
    T, D = 16384, 4096
    g = torch.Generator(device="cuda").manual_seed(5)
    h = torch.empty((T, D), dtype=torch.bfloat16, device="cuda")
    ca, sa, ra = binding.alloc_outputs(T, D, 32, 1)
    cb, sb, rb = binding.alloc_outputs(T, D, 32, 1)
    ct = torch.empty((D, T), dtype=torch.uint8, device="cuda")
    st = torch.empty(binding.scale_bytes(D, T // 32, 1), dtype=torch.uint8, device="cuda")
    ct2, st2 = torch.empty_like(ct), torch.empty_like(st)
    for it in range(12):
        x = (torch.randn(T, D, generator=g, device="cuda") * (1.0 + it)).to(torch.bfloat16)
        res = torch.randn(T, D, generator=g, device="cuda").to(torch.bfloat16)
        torch.cuda.synchronize()
        binding.mxnorm_add_fwd(x, res, h, ca, sa, ra, eps=1e-5, layout=1)      # producer of h (and of its MXNorm)
        binding.mxnorm_fwd(h, None, cb, sb, rb, eps=1e-5, layout=1)            # consumer, launched right behind
        binding.mx_cast_transposed(h, rb, ct, st, eps=1e-5, layout=1)          # second consumer (of h and of rb)
        torch.cuda.synchronize()
        assert torch.equal(ca, cb) and torch.equal(sa, sb) and torch.equal(ra.view(torch.int32), rb.view(torch.int32)), it
        binding.mx_cast_transposed(h, ra, ct2, st2, eps=1e-5, layout=1)        # the same cast with nothing in flight
        torch.cuda.synchronize()
        assert torch.equal(ct, ct2) and torch.equal(st, st2), it
    rows = torch.tensor([0, 1, 4097, T - 1], device="cuda")
    want_c, _, want_r = oracle.mxnorm_ref(wl.bits(h[rows].cpu()), eps=1e-5)
    assert np.array_equal(cb[rows].cpu().numpy(), want_c) and np.array_equal(rb[rows].cpu().numpy(), want_r)
