"""GPU parity of the stand-alone convolution entry point against the oracle (element by element)."""
import numpy as np
import pytest

from harness import rel_err
from oracle import lp_oracle as O
from workloads import gen

pytestmark = pytest.mark.gpu


def run_conv(op, dtype, impl, N, H, W, Cin, Cout, R, stride, pad, a, b, want_stats=False):
    import torch
    import paper_2112_05387_b200 as lp
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    dev = "cuda:0"
    OH, OW = O.out_size(H, R, stride, pad), O.out_size(W, R, stride, pad)
    da = torch.from_numpy(a.astype(np.float32)).to(dev).to(tdt).contiguous()
    if op == lp.LP_CONV_WGRAD:
        db = torch.from_numpy(b.astype(np.float32)).to(dev).to(tdt).contiguous()
        out = torch.full((Cout, R, R, Cin), 7.0, dtype=torch.float32, device=dev)
    else:
        db = torch.from_numpy(b.astype(np.float32)).to(dev).contiguous()
        shape = (N, OH, OW, Cout) if op == lp.LP_CONV_FWD else (N, H, W, Cin)
        out = torch.full(shape, 7.0, dtype=tdt, device=dev)
    nbytes = lp.lp_conv2d_scratch_bytes(Cin, Cout, R)
    scratch = torch.zeros(nbytes + 256, dtype=torch.uint8, device=dev)
    base = (scratch.data_ptr() + 255) // 256 * 256
    stats = torch.zeros(2 * Cout, dtype=torch.float64, device=dev) if want_stats else None
    st, _ = lp.lp_conv2d(op, lp.LP_F32 if dtype == "f32" else lp.LP_BF16, impl, N, H, W, Cin, Cout, R, stride, pad,
                         da, db, out, stats, base, nbytes)
    torch.cuda.synchronize()
    return st, out.float().cpu().numpy().astype(np.float64), (stats.cpu().numpy() if want_stats else None)


def make_case(N, H, W, Cin, Cout, R, stride, pad, dtype, seed=3):
    x = gen.storage_round(gen.normal(seed, "x", (N, H, W, Cin)), dtype).astype(np.float64)
    w = gen.storage_round(gen.normal(seed, "w", (Cout, R, R, Cin), std=(2.0 / (R * R * Cin)) ** 0.5), dtype).astype(np.float64)
    OH, OW = O.out_size(H, R, stride, pad), O.out_size(W, R, stride, pad)
    dy = gen.storage_round(gen.normal(seed, "dy", (N, OH, OW, Cout)), dtype).astype(np.float64)
    return x, w, dy


SIMT_CASES = [
    # N, H, W, Cin, Cout, R, stride, pad
    (2, 8, 8, 3, 8, 3, 1, 1), (2, 8, 8, 8, 8, 3, 1, 1), (3, 9, 7, 8, 16, 3, 2, 1), (2, 8, 8, 8, 16, 1, 2, 0),
    (2, 16, 16, 3, 8, 7, 2, 3),
]


@pytest.mark.parametrize("case", SIMT_CASES)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_simt_conv_matches_oracle(case, dtype):
    import paper_2112_05387_b200 as lp
    N, H, W, Cin, Cout, R, stride, pad = case
    x, w, dy = make_case(*case, dtype)
    tol = 2e-5 if dtype == "f32" else 1e-2
    st, y, stats = run_conv(lp.LP_CONV_FWD, dtype, lp.LP_CONV_IMPL_SIMT, *case, x, w, want_stats=True)
    assert st == 0
    ref = O.conv_fwd(x, w, stride, pad)
    assert rel_err(y, ref) < tol
    # statistics are taken from the stored tensor
    np.testing.assert_allclose(stats[:Cout], y.reshape(-1, Cout).sum(0), rtol=1e-4, atol=1e-3)
    np.testing.assert_allclose(stats[Cout:], (y ** 2).reshape(-1, Cout).sum(0), rtol=1e-4, atol=1e-3)
    if Cin % 4 == 0:
        st, dx, _ = run_conv(lp.LP_CONV_DGRAD, dtype, lp.LP_CONV_IMPL_SIMT, *case, dy, w)
        assert st == 0
        assert rel_err(dx, O.conv_dgrad(dy, w, stride, pad, x.shape)) < tol
    st, dw, _ = run_conv(lp.LP_CONV_WGRAD, dtype, lp.LP_CONV_IMPL_SIMT, *case, x, dy)
    assert st == 0
    assert rel_err(dw, O.conv_wgrad(x, dy, w.shape, stride, pad)) < tol


# tensor-core shapes: several tiles, ragged tails, every swizzle width, strides 1 and 2, 1x1 and 3x3
TC_CASES = [
    (2, 8, 8, 64, 64, 3, 1, 1),       # one tile, 128-byte rows
    (4, 16, 16, 32, 48, 3, 1, 1),     # 64-byte rows, N tile 48
    (3, 32, 32, 16, 16, 3, 1, 1),     # 32-byte rows, ragged batch (3 images of 8 tiles)
    (2, 16, 16, 160, 160, 3, 1, 1),   # wide-ResNet stage-1 channel count (K chunks of 32)
    (5, 8, 8, 320, 320, 3, 1, 1),     # two N tiles of 160, ragged image pairs
    (2, 16, 16, 64, 128, 3, 2, 1),    # stride 2
    (2, 16, 16, 64, 128, 1, 2, 0),    # 1x1 stride-2 projection
    (2, 8, 8, 128, 64, 1, 1, 0),      # 1x1
    (2, 14, 14, 64, 64, 3, 1, 1),     # 14x14: two tile columns, the second ragged
    (3, 7, 7, 128, 128, 3, 1, 1),     # 7x7: one ragged tile column, pairs of images, odd batch
    (2, 32, 32, 40, 160, 3, 1, 1),    # AuxNet hidden width (C_in = 40)
    (2, 32, 32, 160, 80, 3, 2, 1),    # AuxNet strided
    (2, 32, 32, 160, 40, 3, 1, 1),    # AuxNet hidden width as C_out (weight gradient: 32 + 16 channel sub-boxes)
    (32, 32, 32, 64, 64, 3, 1, 1),    # 256 pixel tiles: CTAs work on pairs of tiles sharing the weight stage
    (29, 32, 32, 32, 48, 3, 1, 1),    # 232 tiles: CTAs with one tile and CTAs with a pair
    (64, 16, 16, 32, 320, 3, 1, 1),   # pairs with two channel tiles (ranges cross the channel-tile boundary)
    (37, 16, 16, 160, 160, 3, 2, 1),  # pairs, stride 2, odd tile count (input gradient: parity classes)
    (3, 12, 24, 64, 64, 3, 1, 1),     # 24-wide boxes of 4 rows with a one-row halo, 96 of 128 tile rows used
    (2, 56, 56, 64, 64, 3, 1, 1),     # 56-wide boxes of 2 rows
    (9, 4, 4, 64, 32, 3, 1, 1),       # 4x4 images, eight per tile, ragged last tile
    (40, 32, 32, 160, 160, 3, 1, 1),  # 320 halo tiles of 16x8 pixels: pairs, three K chunks with zero fill
    (5, 12, 20, 64, 256, 3, 1, 1),    # 256-channel tile: eight staging groups, two passes over the accumulator; ragged boxes
    (3, 9, 9, 32, 96, 1, 1, 0),       # odd image size, 81-pixel boxes, three staging groups
    (3, 28, 28, 64, 128, 3, 1, 1),    # width 28: four 8-pixel tile columns, the last one half outside the image
]


# variants of the forward / input-gradient kernel, each forced wherever it applies: tile staged in shared
# memory and stored by TMA; stores from registers; 3x3 stride-1 layers on pairs of CTAs (cta_group::2)
EPILOGUES = {"staged": 512, "direct": 256, "cta-pairs": 1024}   # the last: the CTA-pair kernel where it applies


@pytest.mark.parametrize("epilogue", list(EPILOGUES))
@pytest.mark.parametrize("case", TC_CASES)
def test_tensor_conv_forward_matches_oracle(case, epilogue):
    import paper_2112_05387_b200 as lp
    N, H, W, Cin, Cout, R, stride, pad = case
    x, w, dy = make_case(*case, "bf16")
    st, y, stats = run_conv(lp.LP_CONV_FWD, "bf16", lp.LP_CONV_IMPL_TENSOR | EPILOGUES[epilogue], *case, x, w, want_stats=True)
    assert st == 0, lp.lp_status_string(st)
    ref = O.conv_fwd(x, w, stride, pad)
    assert rel_err(y, ref) < 6e-3
    np.testing.assert_allclose(stats[:Cout], ref.reshape(-1, Cout).sum(0), rtol=1e-3, atol=2e-2 * np.sqrt(ref.size / Cout))
    np.testing.assert_allclose(stats[Cout:], (ref ** 2).reshape(-1, Cout).sum(0), rtol=5e-3)


@pytest.mark.parametrize("epilogue", list(EPILOGUES))
@pytest.mark.parametrize("case", [c for c in TC_CASES if c[3] % 8 == 0 and (c[6] == 1 or (c[1] % 2 == 0 and c[2] % 2 == 0))])
def test_tensor_conv_dgrad_matches_oracle(case, epilogue):
    import paper_2112_05387_b200 as lp
    N, H, W, Cin, Cout, R, stride, pad = case
    x, w, dy = make_case(*case, "bf16")
    st, dx, _ = run_conv(lp.LP_CONV_DGRAD, "bf16", lp.LP_CONV_IMPL_TENSOR | EPILOGUES[epilogue], *case, dy, w)
    assert st == 0, lp.lp_status_string(st)
    assert rel_err(dx, O.conv_dgrad(dy, w, stride, pad, x.shape)) < 6e-3


@pytest.mark.parametrize("case", [c for c in TC_CASES if c[3] % 8 == 0 and c[4] % 8 == 0])
def test_tensor_conv_wgrad_matches_oracle(case):
    import paper_2112_05387_b200 as lp
    N, H, W, Cin, Cout, R, stride, pad = case
    x, w, dy = make_case(*case, "bf16")
    st, dw, _ = run_conv(lp.LP_CONV_WGRAD, "bf16", lp.LP_CONV_IMPL_TENSOR, *case, x, dy)
    assert st == 0, lp.lp_status_string(st)
    assert rel_err(dw, O.conv_wgrad(x, dy, w.shape, stride, pad)) < 2e-3


def test_unsupported_shapes_are_refused_not_faulted():
    import paper_2112_05387_b200 as lp
    case = (2, 8, 8, 3, 8, 3, 1, 1)
    x, w, dy = make_case(*case, "bf16")
    st, _, _ = run_conv(lp.LP_CONV_FWD, "bf16", lp.LP_CONV_IMPL_TENSOR, *case, x, w)
    assert st == -10


@pytest.mark.parametrize("op_name", ["fwd", "dgrad"])
def test_output_on_a_16_byte_boundary_takes_the_narrow_epilogue(op_name):
    """The epilogue writes 32-byte pieces only when the output starts on a 32-byte boundary; a caller
    buffer that is merely 16-byte aligned (the documented requirement) must give the same result."""
    import torch
    import paper_2112_05387_b200 as lp
    case = (4, 16, 16, 64, 64, 3, 1, 1)
    N, H, W, Cin, Cout, R, stride, pad = case
    x, w, dy = make_case(*case, "bf16")
    dev = "cuda:0"
    op = lp.LP_CONV_FWD if op_name == "fwd" else lp.LP_CONV_DGRAD
    a = x if op_name == "fwd" else dy
    da = torch.from_numpy(a.astype(np.float32)).to(dev).to(torch.bfloat16).contiguous()
    dw = torch.from_numpy(w.astype(np.float32)).to(dev).contiguous()
    n_out = N * H * W * (Cout if op_name == "fwd" else Cin)
    nbytes = lp.lp_conv2d_scratch_bytes(Cin, Cout, R)
    scratch = torch.zeros(nbytes + 256, dtype=torch.uint8, device=dev)
    base = (scratch.data_ptr() + 255) // 256 * 256
    results = []
    for shift in (0, 8):                      # elements: 0 -> 256-byte aligned, 8 -> 16 bytes further
        buf = torch.full((n_out + 64,), 7.0, dtype=torch.bfloat16, device=dev)
        off = (-(buf.data_ptr() // 2) % 128) + shift
        out = buf[off:off + n_out]
        assert out.data_ptr() % 32 == (16 if shift else 0)
        st, _ = lp.lp_conv2d(op, lp.LP_BF16, lp.LP_CONV_IMPL_TENSOR, N, H, W, Cin, Cout, R, stride, pad, da, dw, out, None,
                             base, nbytes)
        assert st == 0, lp.lp_status_string(st)
        torch.cuda.synchronize()
        results.append(out.float().cpu().numpy().astype(np.float64))
        assert float(buf[off - 1]) == 7.0 and float(buf[off + n_out]) == 7.0      # nothing written outside
    np.testing.assert_array_equal(results[0], results[1])
    ref = O.conv_fwd(x, w, stride, pad) if op_name == "fwd" else O.conv_dgrad(dy, w, stride, pad, x.shape)
    assert rel_err(results[0], ref.reshape(-1)) < 6e-3
