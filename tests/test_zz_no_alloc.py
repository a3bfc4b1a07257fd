"""The allocation-free forward convolution against the ordinary entry point.

lp_conv2d_fwd_noalloc is for callers that may not allocate device memory (code inside a memory
pool it does not own, a plug-in whose host forbids allocations after start-up, a latency-critical
loop): its scratch is a fixed array inside the library that all calls share and that keeps the
previous call's contents.  The test calls it twice in a row with different shapes -- the second,
smaller call runs over the first one's leftovers -- and compares each result with lp_conv2d on
the same inputs.  This file sorts last so that a run that stops at the first failure has already
run every other test; it also passes when run alone in a fresh process.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _both(case, seed):
    import torch
    import paper_2112_05387_b200 as lp
    N, H, W, Cin, Cout, R, stride, pad = case
    OH, OW = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - R) // stride + 1
    dev = "cuda:0"
    g = torch.Generator(device=dev).manual_seed(seed)
    x = torch.randn(N, H, W, Cin, device=dev, generator=g).to(torch.bfloat16)
    w = (torch.randn(Cout, R, R, Cin, device=dev, generator=g) * (2.0 / (R * R * Cin)) ** 0.5).float()
    # existing entry point: the caller provides the scratch
    y_ref = torch.zeros(N, OH, OW, Cout, device=dev, dtype=torch.bfloat16)
    nbytes = lp.lp_conv2d_scratch_bytes(Cin, Cout, R)
    scratch = torch.zeros(nbytes + 256, dtype=torch.uint8, device=dev)
    base = (scratch.data_ptr() + 255) // 256 * 256
    st, _ = lp.lp_conv2d(lp.LP_CONV_FWD, lp.LP_BF16, lp.LP_CONV_IMPL_TENSOR, N, H, W, Cin, Cout, R, stride, pad,
                         x, w, y_ref, None, base, nbytes)
    assert st == 0, lp.lp_status_string(st)
    # new entry point: inputs and outputs only
    y = torch.full((N, OH, OW, Cout), 3.0, device=dev, dtype=torch.bfloat16)
    st = lp.lp_conv2d_fwd_noalloc(N, H, W, Cin, Cout, R, stride, pad, x, w, y)
    assert st == 0, lp.lp_status_string(st)
    torch.cuda.synchronize()
    a, b = y.float().cpu().numpy().astype(np.float64), y_ref.float().cpu().numpy().astype(np.float64)
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def test_noalloc_forward_matches_lp_conv2d_twice_in_a_row():
    # a large call first, then a smaller one that leaves most of the shared array untouched
    assert _both((4, 16, 16, 320, 320, 3, 1, 1), seed=1) < 6e-3
    assert _both((3, 14, 14, 64, 48, 3, 2, 1), seed=2) < 6e-3
    assert _both((2, 8, 8, 128, 64, 1, 1, 0), seed=3) < 6e-3


def test_noalloc_forward_matches_the_cpu_oracle():
    """One case against the plain definition of the convolution (the oracle), not only against lp_conv2d."""
    import torch
    import paper_2112_05387_b200 as lp
    from oracle import lp_oracle as O
    from workloads import gen
    N, H, W, Cin, Cout, R, stride, pad = 3, 12, 12, 32, 48, 3, 1, 1
    x = gen.round_bf16(gen.normal(11, "x", (N, H, W, Cin)))
    w = gen.round_bf16(gen.normal(11, "w", (Cout, R, R, Cin), std=(2.0 / (R * R * Cin)) ** 0.5))
    dx = torch.from_numpy(x).to("cuda:0").to(torch.bfloat16)
    dw = torch.from_numpy(w).to("cuda:0")
    y = torch.zeros(N, H, W, Cout, device="cuda:0", dtype=torch.bfloat16)
    assert lp.lp_conv2d_fwd_noalloc(N, H, W, Cin, Cout, R, stride, pad, dx, dw, y) == 0
    torch.cuda.synchronize()
    ref = O.conv_fwd(x.astype(np.float64), w.astype(np.float64), stride, pad)
    got = y.float().cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 6e-3


def test_noalloc_rejects_what_does_not_fit_or_is_not_supported():
    import torch
    import paper_2112_05387_b200 as lp
    dev = "cuda:0"
    x = torch.zeros(1, 8, 8, 1024, device=dev, dtype=torch.bfloat16)
    w = torch.zeros(1024, 3, 3, 1024, device=dev, dtype=torch.float32)   # 18.9 MB of bf16 weights > 8 MiB
    y = torch.zeros(1, 8, 8, 1024, device=dev, dtype=torch.bfloat16)
    st = lp.lp_conv2d_fwd_noalloc(1, 8, 8, 1024, 1024, 3, 1, 1, x, w, y)
    assert st == -9 and "size" in lp.lp_status_string(st)
    assert lp.lp_conv2d_fwd_noalloc(1, 8, 8, 3, 8, 3, 1, 1, x, w, y) == -10      # 3 input channels
    assert lp.lp_conv2d_fwd_noalloc(1, 8, 8, 8, 8, 3, 1, 1, None, w, y) == -1
