"""Pins for the oracle's optional storage model (``Net.store``).

The storage model is not part of the paper's method: it states where a reduced-precision implementation
keeps a tensor between two operators, so that the decisions floating point takes (ReLU masks, max-pool
winners) are taken on stored values.  Nothing in the paper fixes it, so the pins are what the model itself
promises:
  * a store that changes nothing leaves every result bit-identical to exact mode (the model adds no
    arithmetic of its own);
  * with a bf16 store, every operand of every contraction (activations, adjoints and the weight operand)
    is a bf16 value, and so is every tensor a block hands to the next one -- a tensor core cannot be
    given anything else;
  * the number of storage points of a module equals the count that follows from the table of stored
    tensors per block kind below (a dropped or added point changes the count);
  * on one-block modules the storage model moves losses by no more than bf16 rounding can, and gradients
    by a few per cent at most.
"""
import numpy as np
import pytest

from conftest import small_cfg
from oracle import lp_oracle as O
from workloads import gen, get_config


def build(cfg):
    net = O.Net(cfg)
    mods = [gen.make_params(net.param_layout(k), cfg["seed"], "module%d" % k, perturb_bn=True, dtype="bf16")
            for k in range(net.K)]
    auxs = [gen.make_params(net.param_layout(O.LP_AUX(k)), cfg["seed"], "aux%d" % k, perturb_bn=True, dtype="bf16")
            for k in range(net.K - 1)]
    x0 = gen.round_bf16(gen.make_images(cfg)).astype(np.float64)
    xs = [x0] + [gen.round_bf16(x).astype(np.float64) for x in O.auxnet_forward(net, auxs, x0)]
    return net, mods, auxs, xs, gen.make_labels(cfg)


def run_modules(net, mods, xs, labels, rho, store, kappa_std=0.3):
    net.store = store
    try:
        out = []
        for k in range(net.K):
            last = k == net.K - 1
            kap = None if last else gen.round_bf16(gen.normal(5, "kap%d" % k, xs[k + 1].shape, std=kappa_std)).astype(np.float64)
            out.append(O.module_fwd_bwd(net, k, mods[k], xs[k], labels if last else xs[k + 1], kap, rho))
        return out
    finally:
        net.store = None


SHAPES = [
    ("tiny", lambda: get_config("tiny")),
    ("postbn", lambda: small_cfg("postbn", stage_blocks=(2, 2), module_block_end=(1, 3, 4), N=3)),
    ("postbn-7x7", lambda: small_cfg("postbn", stem="conv7x7s2_maxpool", H=16, W=16, N=3, stage_channels=(8, 8),
                                     stage_stride=(1, 1))),
    ("preact", lambda: small_cfg("preact", stage_blocks=(2, 2), module_block_end=(1, 3, 4), N=3)),
    ("preact-K1", lambda: small_cfg("preact", module_block_end=(2,), N=3)),
    ("bottleneck", lambda: small_cfg("bottleneck", stage_channels=(16, 32), stage_blocks=(2, 2),
                                     module_block_end=(1, 3, 4), N=3, stem_channels=16)),
]


def is_bf16(a):
    a = np.asarray(a, dtype=np.float64)
    return np.array_equal(a, gen.round_bf16(a).astype(np.float64))


# ---------------------------------------------------------------------------------------------
# a store that changes nothing changes nothing
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name,mk", SHAPES)
def test_identity_store_is_bit_identical_to_exact_mode(name, mk):
    cfg = mk()
    net, mods, auxs, xs, labels = build(cfg)
    exact = run_modules(net, mods, xs, labels, cfg["rho"], None)
    ident = run_modules(net, mods, xs, labels, cfg["rho"], lambda a: a)
    for k in range(net.K):
        assert exact[k]["loss"] == ident[k]["loss"]
        np.testing.assert_array_equal(exact[k]["grads"], ident[k]["grads"])
        if k > 0:
            np.testing.assert_array_equal(exact[k]["dx"], ident[k]["dx"])
        if k < net.K - 1:
            np.testing.assert_array_equal(exact[k]["seed"], ident[k]["seed"])
    # AuxNet chain, its distillation pass and the recursive stacks
    x0 = xs[0]
    a = O.auxnet_forward(net, auxs, x0)
    net.store = lambda v: v
    b = O.auxnet_forward(net, auxs, x0)
    net.store = None
    for u, v in zip(a, b):
        np.testing.assert_array_equal(u, v)
    if net.K > 1:
        tgt = a[0] + 0.1
        r0 = O.auxnet_fwd_bwd(net, 0, auxs[0], x0, tgt)
        net.store = lambda v: v
        r1 = O.auxnet_fwd_bwd(net, 0, auxs[0], x0, tgt)
        net.store = None
        assert r0["loss"] == r1["loss"]
        np.testing.assert_array_equal(r0["grads"], r1["grads"])


# ---------------------------------------------------------------------------------------------
# with a bf16 store every contraction operand and every tensor kept between blocks is a bf16 value
# ---------------------------------------------------------------------------------------------
class OperandRecorder:
    """Wraps the oracle's three contractions and records whether their operands are bf16 values."""

    def __init__(self, monkeypatch):
        self.bad, self.calls = [], 0
        for name in ("conv_fwd", "conv_dgrad", "conv_wgrad"):
            orig = getattr(O, name)
            monkeypatch.setattr(O, name, self.wrap(name, orig))

    def wrap(self, name, orig):
        def f(a, b, *rest):
            self.calls += 1
            for i, t in enumerate((a, b)):
                if not is_bf16(t):
                    self.bad.append((name, i, np.asarray(t).shape))
            return orig(a, b, *rest)
        return f


@pytest.mark.parametrize("name,mk", SHAPES)
def test_bf16_store_makes_every_contraction_operand_a_bf16_value(name, mk, monkeypatch):
    cfg = mk()
    net, mods, auxs, xs, labels = build(cfg)
    rec = OperandRecorder(monkeypatch)
    res = run_modules(net, mods, xs, labels, cfg["rho"], gen.round_bf16)
    assert rec.calls > 0 and not rec.bad, rec.bad
    for k in range(net.K):
        if k > 0:
            assert is_bf16(res[k]["dx"]), ("dx", k)           # what the step hands to the caller
        if k < net.K - 1:
            assert is_bf16(res[k]["r"]), ("r", k)
    # AuxNet chain forward and distillation backward, recursive stacks
    rec.calls, rec.bad = 0, []
    net.store = gen.round_bf16
    try:
        ax = O.auxnet_forward(net, auxs, xs[0])
        for k in range(net.K - 1):
            assert is_bf16(ax[k]), ("x", k + 1)
            x_in = xs[0] if k == 0 else ax[k - 1]
            O.auxnet_fwd_bwd(net, k, auxs[k], x_in, ax[k] + gen.round_bf16(gen.normal(9, "t%d" % k, ax[k].shape, std=0.1)))
        if net.K > 2:
            stacks = [[auxs[j] for j in range(k)] for k in range(1, net.K)]
            rx = O.reauxnet_forward(net, stacks, xs[0])
            O.reauxnet_fwd_bwd(net, net.K - 1, stacks[-1], xs[0], rx[-1] + 0.125)
    finally:
        net.store = None
    assert (rec.calls > 0 or net.K == 1) and not rec.bad, rec.bad


def test_a_store_that_is_skipped_is_noticed_by_the_operand_check(monkeypatch):
    """The check above has teeth: a storage model that leaves one kind of tensor unrounded (here every
    second call passes its argument through) is reported."""
    cfg = small_cfg("preact", N=3)
    net, mods, auxs, xs, labels = build(cfg)
    rec = OperandRecorder(monkeypatch)
    n = [0]

    def leaky(a):
        n[0] += 1
        return a if n[0] % 2 else gen.round_bf16(a)
    run_modules(net, mods, xs, labels, cfg["rho"], leaky)
    assert rec.bad


# ---------------------------------------------------------------------------------------------
# number of storage points per module
# ---------------------------------------------------------------------------------------------
# Tensors a module keeps, per part (activation / adjoint tensors written to memory, and the reduced-
# precision operand copy of the weights, once per contraction that reads it):
#   stem, post-BN nets     forward  w, y, a = relu(bn(y))                 backward  dy            (+ d(pool) with max-pool)
#   stem, pre-act net      forward  w, y                                  backward  -
#   post-BN block          forward  w1, y1, a1, w2, y2 (+ ws, ys)         backward  dy2, w2, da1, dy1, w1, dx (+ dys, dx', ws)
#   bottleneck block       forward  w1, y1, a1, w2, y2, a2, w3, y3 (+ ws, ys)
#                          backward dy3, w3, da2, dy2, w2, da1, dy1, w1, dx (+ dys, dx', ws)
#   pre-act block          forward  o = relu(bn(x)), w1, y1, a1, w2 (+ ws, ys), out
#                          backward w2, da1, dy1, w1, do, dx (+ ws, do')
#   block output           post-BN / bottleneck nets: kept, except for the last block of an interior module,
#                          whose output goes straight into the local loss in full precision
#   local loss             r, terminal adjoint
#   head                   post-BN nets: backward d(pool);  pre-act net: forward relu(bn(x)), backward d(pool), dx of the BN
POINTS = {
    "postbn": dict(stem=3 + 1, pool=1, fwd=5, fwd_proj=2, bwd=6, bwd_proj=3, head=1),
    "bottleneck": dict(stem=3 + 1, pool=1, fwd=8, fwd_proj=2, bwd=9, bwd_proj=3, head=1),
    "preact": dict(stem=2, pool=0, fwd=5 + 1, fwd_proj=2, bwd=6, bwd_proj=2, head=3),
}


def expected_points(net, k):
    t = POINTS[net.kind]
    n = 0
    if k == 0:
        n += t["stem"] + (t["pool"] if net.stem["pool"] else 0)
    blocks = net.module_blocks[k]
    for i, bi in enumerate(blocks):
        proj = net.blocks[bi]["proj"]
        n += t["fwd"] + t["bwd"] + (t["fwd_proj"] + t["bwd_proj"] if proj else 0)
        if net.post and not (i == len(blocks) - 1 and k < net.K - 1):
            n += 1                                   # block output kept
    n += t["head"] if k == net.K - 1 else 2          # head, or r and the terminal adjoint
    return n


@pytest.mark.parametrize("name,mk", SHAPES)
def test_number_of_storage_points_follows_the_table(name, mk):
    cfg = mk()
    net, mods, auxs, xs, labels = build(cfg)
    for k in range(net.K):
        calls = [0]

        def store(a):
            calls[0] += 1
            return a
        net.store = store
        last = k == net.K - 1
        O.module_fwd_bwd(net, k, mods[k], xs[k], labels if last else xs[k + 1], None if last else np.zeros_like(xs[k + 1]),
                         cfg["rho"])
        net.store = None
        assert calls[0] == expected_points(net, k), (k, calls[0], expected_points(net, k))


def test_storage_points_of_an_auxnet_unit():
    """AuxNet (conv-BN-ReLU-conv-BN): forward w1, y1, h, w2, y2, out; distillation backward seed, dy2, w2, dh, dy1."""
    cfg = small_cfg("preact", N=3)
    net, mods, auxs, xs, labels = build(cfg)
    calls = [0]

    def store(a):
        calls[0] += 1
        return a
    net.store = store
    O.auxnet_forward(net, auxs, xs[0])
    fwd = calls[0]
    calls[0] = 0
    O.auxnet_fwd_bwd(net, 0, auxs[0], xs[0], xs[1])
    net.store = None
    assert fwd == 6 and calls[0] == 6 + 5


# ---------------------------------------------------------------------------------------------
# size of the effect
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("kind", ["postbn", "preact", "bottleneck"])
@pytest.mark.parametrize("N,H", [(6, 8), (16, 16)])
def test_storage_model_stays_within_bf16_rounding_of_exact_arithmetic_on_one_block_modules(kind, N, H):
    """One block per module.  The forward quantities move by rounding only: losses within 2e-3 of exact
    arithmetic (seen: 3e-6 .. 3e-4).  Gradients also feel the ReLU masks that flip where a pre-activation
    lies within rounding of zero: the whole-module gradient moves by 0.3 % .. 3 % (seen over these shapes),
    so the bound here is 5e-2 -- already a one-block module cannot be held to 2e-2 against exact arithmetic,
    which is why gradients of bf16 workloads are compared with the storage model on both sides."""
    ch = (16, 32) if kind == "bottleneck" else (8, 16)
    cfg = small_cfg(kind, N=N, H=H, W=H, stage_channels=ch, stage_blocks=(1, 1), module_block_end=(1, 2), stem_channels=ch[0])
    net, mods, auxs, xs, labels = build(cfg)
    exact = run_modules(net, mods, xs, labels, cfg["rho"], None)
    stored = run_modules(net, mods, xs, labels, cfg["rho"], gen.round_bf16)
    for k in range(net.K):
        assert abs(stored[k]["loss"] - exact[k]["loss"]) < 2e-3 * abs(exact[k]["loss"])
        e = np.linalg.norm(stored[k]["grads"] - exact[k]["grads"]) / np.linalg.norm(exact[k]["grads"])
        assert 0 < e < 5e-2, (k, e)                  # moved (the model does round something), but by little
