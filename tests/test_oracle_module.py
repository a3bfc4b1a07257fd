"""Pins for the oracle's module forward/backward, local losses, AuxNet chain and step.

The paper prints no worked numeric example, so the pins are the facts it does fix:
  (ii)  local back-propagation is the ordinary gradient of the local loss -> finite differences;
  (iii) the penalty vanishes on the feasible set (psi(x, x) = 0): loss and all gradients are zero;
  (iv)  kappa = 0 turns the augmented-Lagrangian method into the penalty method; the AL terms are
        linear in kappa;
  (v)   with consistent auxiliary variables the K modules reproduce the layer-serial network.
A PyTorch-CPU autograd run on a tiny network is a secondary, library-based cross-check.
"""
import numpy as np
import pytest

from conftest import small_cfg
from oracle import lp_oracle as O
from workloads import gen, get_config


def build(cfg, perturb=True):
    net = O.Net(cfg)
    mods = [gen.make_params(net.param_layout(k), cfg["seed"], "module%d" % k, perturb_bn=perturb)
            for k in range(net.K)]
    auxs = [gen.make_params(net.param_layout(O.LP_AUX(k)), cfg["seed"], "aux%d" % k, perturb_bn=perturb)
            for k in range(net.K - 1)]
    return net, mods, auxs


ALL_CFGS = [
    ("tiny", lambda: get_config("tiny")),
    ("postbn-proj", lambda: small_cfg("postbn")),
    ("preact-proj", lambda: small_cfg("preact")),
    ("postbn-7x7", lambda: small_cfg("postbn", stem="conv7x7s2_maxpool", H=16, W=16, N=3,
                                     stage_channels=(8, 8), stage_stride=(1, 1))),
    ("preact-3mod", lambda: small_cfg("preact", stage_channels=(8, 16), stage_blocks=(2, 2),
                                      module_block_end=(1, 3, 4), N=3)),
    # bottleneck blocks (1x1 - 3x3 - 1x1, the block of the paper's ResNet-50 workload): identity and
    # projection shortcuts, a stride-2 block, a module boundary inside a stage
    ("bottleneck", lambda: small_cfg("bottleneck", stage_channels=(16, 32), stage_blocks=(2, 2),
                                     module_block_end=(1, 3, 4), N=3, stem_channels=16)),
]


@pytest.mark.parametrize("name,mk", ALL_CFGS)
def test_layouts_and_shapes(name, mk):
    cfg = mk()
    net, mods, auxs = build(cfg)
    x = gen.make_images(cfg)
    xs = O.auxnet_forward(net, auxs, x)
    assert len(xs) == net.K - 1
    for k in range(1, net.K):
        assert xs[k - 1].shape == net.boundary[k]
    for k in range(net.K - 1):
        out = O.module_forward(net, k, net.unpack(k, mods[k]), x if k == 0 else xs[k - 1])
        assert out.shape == net.boundary[k + 1]
    for k in range(net.K):
        assert mods[k].size == net.param_count(k)


@pytest.mark.parametrize("name,mk", ALL_CFGS)
def test_ii_finite_difference_gradients(name, mk):
    cfg = mk()
    net, mods, auxs = build(cfg)
    x0 = gen.make_images(cfg).astype(np.float64)
    xs = [x0] + O.auxnet_forward(net, auxs, x0)
    labels = gen.make_labels(cfg)
    rho = cfg["rho"]
    for k in range(net.K):
        last = k == net.K - 1
        tgt = labels if last else xs[k + 1]
        kap = None if last else gen.normal(5, "kap%d" % k, xs[k + 1].shape, std=0.3)
        res = O.module_fwd_bwd(net, k, mods[k], xs[k], tgt, kap, rho)
        p0 = mods[k].astype(np.float64)

        def loss_of_params(p):
            out = O.module_forward(net, k, net.unpack(k, p), xs[k])
            return O.softmax_ce(out, labels)[0] if last else O.local_loss(out, tgt, kap, rho)[0]

        def loss_of_x(xx):
            out = O.module_forward(net, k, net.unpack(k, p0), xx)
            return O.softmax_ce(out, labels)[0] if last else O.local_loss(out, tgt, kap, rho)[0]

        # sample parameters from every tensor of the layout
        off = 0
        scale = max(1.0, abs(res["loss"]))
        for pname, _, shape in net.param_layout(k):
            n = int(np.prod(shape))
            for j in sorted(set([off, off + n // 2, off + n - 1])):
                h = 1e-5
                pp, pm = p0.copy(), p0.copy()
                pp[j] += h
                pm[j] -= h
                fd = (loss_of_params(pp) - loss_of_params(pm)) / (2 * h)
                assert abs(fd - res["grads"][j]) < 2e-6 * scale + 1e-5 * abs(fd), (name, k, pname, j, fd, res["grads"][j])
            off += n
        if k > 0:
            flat = xs[k].reshape(-1)
            for j in [0, flat.size // 3, flat.size - 1]:
                h = 1e-5
                xp, xm = flat.copy(), flat.copy()
                xp[j] += h
                xm[j] -= h
                fd = (loss_of_x(xp.reshape(xs[k].shape)) - loss_of_x(xm.reshape(xs[k].shape))) / (2 * h)
                assert abs(fd - res["dx"].reshape(-1)[j]) < 2e-6 * scale + 1e-5 * abs(fd)
        else:
            assert res["dx"] is None


@pytest.mark.parametrize("name,mk", ALL_CFGS)
def test_iii_penalty_vanishes_on_feasible_set(name, mk):
    cfg = mk()
    net, mods, auxs = build(cfg)
    x0 = gen.make_images(cfg).astype(np.float64)
    xs = [x0] + O.auxnet_forward(net, auxs, x0)
    for k in range(net.K - 1):
        feasible = O.module_forward(net, k, net.unpack(k, mods[k]), xs[k])
        res = O.module_fwd_bwd(net, k, mods[k], xs[k], feasible, None, 3.0)
        assert res["loss"] == 0.0 and res["rnorm2"] == 0.0
        assert np.all(res["grads"] == 0.0)
        assert res["dx"] is None or np.all(res["dx"] == 0.0)


@pytest.mark.parametrize("name,mk", ALL_CFGS[:3])
def test_iv_al_reduces_to_penalty_and_is_linear_in_kappa(name, mk):
    cfg = mk()
    net, mods, auxs = build(cfg)
    x0 = gen.make_images(cfg).astype(np.float64)
    xs = [x0] + O.auxnet_forward(net, auxs, x0)
    rho = 0.8
    for k in range(net.K - 1):
        tgt = xs[k + 1]
        pen = O.module_fwd_bwd(net, k, mods[k], xs[k], tgt, None, rho)
        al0 = O.module_fwd_bwd(net, k, mods[k], xs[k], tgt, np.zeros_like(tgt), rho)
        assert al0["loss"] == pen["loss"]
        np.testing.assert_array_equal(al0["grads"], pen["grads"])
        np.testing.assert_array_equal(al0["seed"], pen["seed"])
        kap = gen.normal(9, "k", tgt.shape, std=0.2)
        al1 = O.module_fwd_bwd(net, k, mods[k], xs[k], tgt, kap, rho)
        al2 = O.module_fwd_bwd(net, k, mods[k], xs[k], tgt, 2 * kap, rho)
        assert abs((al1["loss"] - pen["loss"]) - float((kap * pen["r"]).sum())) < 1e-9 * max(1, abs(pen["loss"]))
        d1 = al1["grads"] - pen["grads"]
        d2 = al2["grads"] - pen["grads"]
        np.testing.assert_allclose(d2, 2 * d1, rtol=1e-8, atol=1e-9 * np.abs(pen["grads"]).max())
        # terminal adjoint: rho*r + kappa; with the multiplier step c = rho the new kappa equals it
        np.testing.assert_allclose(al1["seed"], rho * al1["r"] + kap, rtol=1e-14)
        np.testing.assert_allclose(O.kappa_update(kap, al1["r"], rho), al1["seed"], rtol=1e-14, atol=1e-15)


@pytest.mark.parametrize("name,mk", ALL_CFGS)
def test_v_consistent_chain_reproduces_layer_serial_network(name, mk):
    cfg = mk()
    net, mods, auxs = build(cfg)
    x0 = gen.make_images(cfg).astype(np.float64)
    x = x0
    for k in range(net.K):
        x = O.module_forward(net, k, net.unpack(k, mods[k]), x)      # x_{k+1} := F_k(x_k)
    serial = O.forward_serial(net, mods, x0)
    np.testing.assert_allclose(x, serial, rtol=1e-11, atol=1e-12)


def test_identity_blocks_pass_features_through():
    """Zero conv weights make F(X, W) = 0 in the pre-activation block, so X_{l+1} = X_l."""
    cfg = small_cfg("preact", stage_channels=(8, 8), stage_stride=(1, 1), module_block_end=(1, 2))
    net, mods, auxs = build(cfg)
    named = net.unpack(1, mods[1])
    named = {n: (np.zeros_like(v) if n.endswith("conv2.w") else v) for n, v in named.items()}
    x1 = gen.normal(2, "x1", net.boundary[1])
    c = {}
    y = x1
    for bi in net.module_blocks[1]:
        y = O._block_fwd(net, bi, named, y, c)
    np.testing.assert_array_equal(y, x1)


def test_last_module_zero_head_gives_log_classes():
    cfg = get_config("tiny")
    net, mods, auxs = build(cfg)
    named = net.unpack(1, mods[1])
    named["head.fc.w"] = np.zeros_like(named["head.fc.w"])
    named["head.fc.b"] = np.zeros_like(named["head.fc.b"])
    x1 = gen.normal(2, "x1", net.boundary[1])
    res = O.module_fwd_bwd(net, 1, net.pack(1, named), x1, gen.make_labels(cfg), None, 1.0)
    assert abs(res["loss"] - np.log(10)) < 1e-12


def test_step_two_updates_closed_form():
    cfg = get_config("tiny")
    net, mods, auxs = build(cfg)
    x0 = gen.make_images(cfg)
    labels = gen.make_labels(cfg)
    kap = [gen.make_kappa(cfg, 0, net.boundary[1])]
    newp, newk, results, xs = O.layer_parallel_step(net, mods, auxs, x0, labels, kap, 1.0, 0.1)
    for k in range(net.K):
        np.testing.assert_allclose(newp[k], mods[k] - 0.1 * results[k]["grads"], rtol=1e-15)
    np.testing.assert_allclose(newk[0], results[0]["seed"], rtol=1e-13, atol=1e-15)
    # a second step starts from the updated multiplier: the loss gains <kappa_new, r_new>
    newp2, newk2, results2, _ = O.layer_parallel_step(net, newp, auxs, x0, labels, newk, 1.0, 0.1)
    pen2 = O.module_fwd_bwd(net, 0, newp[0], x0, xs[1], None, 1.0)
    assert abs(results2[0]["loss"] - pen2["loss"] - float((newk[0] * pen2["r"]).sum())) < 1e-9


def test_torch_autograd_crosscheck():
    """Secondary pin: PyTorch CPU autograd on a post-activation and a pre-activation module."""
    torch = pytest.importorskip("torch")
    import torch.nn.functional as Fn
    for kind in ("postbn", "preact"):
        cfg = small_cfg(kind)
        net, mods, auxs = build(cfg)
        k = 1
        x = gen.normal(4, "x", net.boundary[1])
        labels = gen.make_labels(cfg)
        res = O.module_fwd_bwd(net, k, mods[k], x, labels, None, 1.0)
        named = {n: torch.tensor(v, dtype=torch.float64, requires_grad=True)
                 for n, v in net.unpack(k, mods[k]).items()}
        xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)

        def conv(t, w, stride, pad):
            return Fn.conv2d(t.permute(0, 3, 1, 2), w.permute(0, 3, 1, 2), stride=stride, padding=pad).permute(0, 2, 3, 1)

        def bn(t, g, b):
            return Fn.batch_norm(t.permute(0, 3, 1, 2), None, None, g, b, True, 0.0, cfg["bn_eps"]).permute(0, 2, 3, 1)

        h = xt
        for bi in net.module_blocks[k]:
            b = net.blocks[bi]
            q = "block%d." % bi
            if kind == "postbn":
                t = torch.relu(bn(conv(h, named[q + "conv1.w"], b["stride"], 1), named[q + "bn1.g"], named[q + "bn1.b"]))
                t = bn(conv(t, named[q + "conv2.w"], 1, 1), named[q + "bn2.g"], named[q + "bn2.b"])
                s = bn(conv(h, named[q + "sc.w"], b["stride"], 0), named[q + "bns.g"], named[q + "bns.b"]) if b["proj"] else h
            else:
                o = torch.relu(bn(h, named[q + "bn1.g"], named[q + "bn1.b"]))
                t = torch.relu(bn(conv(o, named[q + "conv1.w"], b["stride"], 1), named[q + "bn2.g"], named[q + "bn2.b"]))
                t = conv(t, named[q + "conv2.w"], 1, 1)
                s = conv(o, named[q + "sc.w"], b["stride"], 0) if b["proj"] else h
            h = s + t
        if kind == "preact":
            h = torch.relu(bn(h, named["head.bn.g"], named["head.bn.b"]))
        logits = h.mean(dim=(1, 2)) @ named["head.fc.w"].T + named["head.fc.b"]
        loss = Fn.cross_entropy(logits, torch.tensor(labels, dtype=torch.long))
        loss.backward()
        assert abs(loss.item() - res["loss"]) < 1e-10
        tg = net.pack(k, {n: v.grad.numpy() for n, v in named.items()})
        np.testing.assert_allclose(res["grads"], tg, rtol=1e-7, atol=1e-10)
        np.testing.assert_allclose(res["dx"], xt.grad.numpy(), rtol=1e-7, atol=1e-12)


# -- AuxNet correction and distillation (second loop of Algorithm 1) ---------------------------
@pytest.mark.parametrize("name,mk", ALL_CFGS[:3] + ALL_CFGS[4:])
def test_auxnet_distillation_gradients(name, mk):
    cfg = mk()
    net, mods, auxs = build(cfg)
    x0 = gen.make_images(cfg).astype(np.float64)
    xs = [x0] + O.auxnet_forward(net, auxs, x0)
    for k in range(net.K - 1):
        target = xs[k + 1] + 0.3 * gen.normal(8, "t%d" % k, xs[k + 1].shape)
        res = O.auxnet_fwd_bwd(net, k, auxs[k], xs[k], target)
        np.testing.assert_allclose(res["out"], xs[k + 1], rtol=1e-12, atol=1e-12)     # same forward as the chain
        assert abs(res["loss"] - float(((xs[k + 1] - target) ** 2).sum())) < 1e-9 * res["loss"]
        p0 = auxs[k].astype(np.float64)

        def loss_of(p):
            out = O.auxnet_apply(net, k, net.unpack(O.LP_AUX(k), p), xs[k])
            return float(((out - target) ** 2).sum())
        off = 0
        for pname, _, shape in net.param_layout(O.LP_AUX(k)):
            n = int(np.prod(shape))
            for j in sorted(set([off, off + n // 2, off + n - 1])):
                h = 1e-5
                pp, pm = p0.copy(), p0.copy()
                pp[j] += h
                pm[j] -= h
                fd = (loss_of(pp) - loss_of(pm)) / (2 * h)
                assert abs(fd - res["grads"][j]) < 2e-6 * max(1.0, res["loss"]) + 1e-5 * abs(fd), (name, k, pname, j)
            off += n
        # the target reproduced exactly: zero loss, zero gradients
        zero = O.auxnet_fwd_bwd(net, k, auxs[k], xs[k], xs[k + 1])
        assert zero["loss"] == 0.0 and np.all(zero["grads"] == 0.0)


def test_aux_correction_direction_and_distillation_is_linear_in_the_step():
    """g_k = P^k_{kn} + rho (x_k - out_{k-1}) - kappa_k = dx_k - seed_{k-1}; the distillation gradient
    for the target x_k - lr*g_k is 2*lr*J^T g_k, linear in lr."""
    cfg = get_config("tiny")
    net, mods, auxs = build(cfg)
    x0 = gen.make_images(cfg).astype(np.float64)
    xs = [x0] + O.auxnet_forward(net, auxs, x0)
    labels = gen.make_labels(cfg)
    rho = 0.7
    kap = gen.normal(3, "kap", xs[1].shape, std=0.2)
    r0 = O.module_fwd_bwd(net, 0, mods[0], xs[0], xs[1], kap, rho)
    r1 = O.module_fwd_bwd(net, 1, mods[1], xs[1], labels, None, rho)
    x_new, g = O.aux_correction(xs[1], r1["dx"], r0["seed"], 0.05)
    np.testing.assert_allclose(g, r1["dx"] + rho * (xs[1] - r0["out"]) - kap, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(x_new, xs[1] - 0.05 * g, rtol=1e-14)
    g1 = O.auxnet_fwd_bwd(net, 0, auxs[0], x0, xs[1] - 0.05 * g)["grads"]
    g2 = O.auxnet_fwd_bwd(net, 0, auxs[0], x0, xs[1] - 0.10 * g)["grads"]
    np.testing.assert_allclose(g2, 2 * g1, rtol=1e-9, atol=1e-12)
    newp, newx, losses, grads = O.auxnet_distill_step(net, auxs, x0, xs[1:], [r1["dx"]], [r0["seed"]], 0.05, 0.01)
    np.testing.assert_allclose(grads[0], g1, rtol=1e-12)
    np.testing.assert_allclose(newp[0], auxs[0] - 0.01 * g1, rtol=1e-12, atol=1e-15)
    assert abs(losses[0] - 0.05 ** 2 * float((g * g).sum())) < 1e-12 * max(1.0, losses[0])


# -- Recursive auxiliary-variable networks (Eq. ReAuxNet-FP, Eq. ReAuxNet-Distill) ------------------
def build_stacks(net, cfg, perturb=True):
    """Stack k (k = 1..K-1) holds k units with parameters of their own; unit j has AuxNet_j's layout."""
    return [[gen.make_params(net.param_layout(O.LP_AUX(j)), cfg["seed"], "reaux%d/%d" % (k, j), perturb_bn=perturb)
             for j in range(k)] for k in range(1, net.K)]


REAUX_CFGS = [ALL_CFGS[4],
              ("postbn-4mod", lambda: small_cfg("postbn", stage_channels=(8, 16), stage_blocks=(2, 2),
                                                module_block_end=(1, 2, 3, 4), N=3))]


@pytest.mark.parametrize("name,mk", REAUX_CFGS)
def test_reauxnet_with_shared_first_parts_is_the_auxnet_chain(name, mk):
    """The paper's remark at the end of the section: stacks whose leading units share the chain's
    parameters degenerate to the serial AuxNet chain; and for k = 1 the stack is AuxNet_0 itself."""
    cfg = mk()
    net, mods, auxs = build(cfg)
    x0 = gen.make_images(cfg).astype(np.float64)
    chain = O.auxnet_forward(net, auxs, x0)
    shared = [[auxs[j] for j in range(k)] for k in range(1, net.K)]
    rec = O.reauxnet_forward(net, shared, x0)
    assert len(rec) == net.K - 1
    for a, b in zip(rec, chain):
        np.testing.assert_array_equal(a, b)
    target = chain[0] + 0.2 * gen.normal(5, "t", chain[0].shape)
    r1 = O.reauxnet_fwd_bwd(net, 1, shared[0], x0, target)
    r2 = O.auxnet_fwd_bwd(net, 0, auxs[0], x0, target)
    assert r1["loss"] == r2["loss"]
    np.testing.assert_array_equal(r1["grads"][0], r2["grads"])
    # independent parameters give different variables, each of its boundary's shape
    stacks = build_stacks(net, cfg)
    own = O.reauxnet_forward(net, stacks, x0)
    for k in range(1, net.K):
        assert own[k - 1].shape == tuple(net.boundary[k])
    assert not np.allclose(own[-1], chain[-1])


@pytest.mark.parametrize("name,mk", REAUX_CFGS)
def test_reauxnet_distillation_gradients_by_finite_differences(name, mk):
    cfg = mk()
    net, mods, auxs = build(cfg)
    stacks = build_stacks(net, cfg)
    x0 = gen.make_images(cfg).astype(np.float64)
    xs = O.reauxnet_forward(net, stacks, x0)
    for k in range(1, net.K):
        target = xs[k - 1] + 0.3 * gen.normal(9, "t%d" % k, xs[k - 1].shape)
        res = O.reauxnet_fwd_bwd(net, k, stacks[k - 1], x0, target)
        np.testing.assert_allclose(res["out"], xs[k - 1], rtol=1e-12, atol=1e-12)
        assert len(res["grads"]) == k

        def loss_of(j, p):
            st = list(stacks[k - 1])
            st[j] = p
            out = _stack_forward(net, k, st, x0)
            return float(((out - target) ** 2).sum())
        for j in range(k):
            p0 = stacks[k - 1][j].astype(np.float64)
            off = 0
            for pname, _, shape in net.param_layout(O.LP_AUX(j)):
                n = int(np.prod(shape))
                for i in sorted(set([off, off + n // 2, off + n - 1])):
                    h = 1e-5
                    pp, pm = p0.copy(), p0.copy()
                    pp[i] += h
                    pm[i] -= h
                    fd = (loss_of(j, pp) - loss_of(j, pm)) / (2 * h)
                    assert abs(fd - res["grads"][j][i]) < 2e-6 * max(1.0, res["loss"]) + 1e-5 * abs(fd), (name, k, j, pname, i)
                off += n
        zero = O.reauxnet_fwd_bwd(net, k, stacks[k - 1], x0, xs[k - 1])
        assert zero["loss"] == 0.0 and all(np.all(g == 0.0) for g in zero["grads"])


def _stack_forward(net, k, stack, x0):
    """Stack k alone, written with the chain's own unit function (not the stack code under test)."""
    x = np.asarray(x0, dtype=np.float64)
    for j in range(k):
        x = O.auxnet_apply(net, j, net.unpack(O.LP_AUX(j), stack[j]), x)
    return x


def test_reauxnet_distill_step_closed_form():
    """One distillation step: x_k_new = x_k - lr*(dx_k - seed_{k-1}); since x_k was just generated by
    the stack, the loss is lr^2 ||g_k||^2 and the gradient is linear in lr; units take plain SGD steps."""
    cfg = REAUX_CFGS[0][1]()
    net, mods, auxs = build(cfg)
    stacks = build_stacks(net, cfg)
    x0 = gen.make_images(cfg).astype(np.float64)
    xs = O.reauxnet_forward(net, stacks, x0)
    dxs = [gen.normal(11, "dx%d" % k, xs[k - 1].shape, std=0.1) for k in range(1, net.K)]
    seeds = [gen.normal(12, "sd%d" % k, xs[k - 1].shape, std=0.1) for k in range(1, net.K)]
    new1, newx1, loss1, g1 = O.reauxnet_distill_step(net, stacks, x0, xs, dxs, seeds, 0.05, 0.01)
    new2, newx2, loss2, g2 = O.reauxnet_distill_step(net, stacks, x0, xs, dxs, seeds, 0.10, 0.01)
    for k in range(1, net.K):
        g = dxs[k - 1] - seeds[k - 1]
        np.testing.assert_allclose(newx1[k - 1], xs[k - 1] - 0.05 * g, rtol=1e-14)
        assert abs(loss1[k - 1] - 0.05 ** 2 * float((g * g).sum())) < 1e-10 * max(1.0, loss1[k - 1])
        for j in range(k):
            np.testing.assert_allclose(g2[k - 1][j], 2 * g1[k - 1][j], rtol=1e-8, atol=1e-12)
            np.testing.assert_allclose(new1[k - 1][j], stacks[k - 1][j] - 0.01 * g1[k - 1][j], rtol=1e-12, atol=1e-15)


def test_bottleneck_shift_before_1x1_convolutions_and_batch_norms_has_no_gradient():
    """A per-channel shift of a tensor that only feeds 1x1 convolutions followed by batch norms is
    removed by their mean subtraction: the local loss does not depend on bn3.beta of a bottleneck block
    whose successor has a projection shortcut (3x3 convolutions do see it, through their zero padding)."""
    cfg = ALL_CFGS[5][1]()
    net, mods, auxs = build(cfg)
    x0 = gen.make_images(cfg).astype(np.float64)
    xs = [x0] + O.auxnet_forward(net, auxs, x0)
    k = 1                                         # blocks 1 (identity shortcut) and 2 (projection, stride 2)
    assert net.module_blocks[k] == [1, 2] and net.blocks[2]["proj"]
    res = O.module_fwd_bwd(net, k, mods[k], xs[k], xs[k + 1], None, 0.7)
    g = net.unpack(k, res["grads"])
    scale = np.linalg.norm(res["grads"])
    assert np.linalg.norm(g["block1.bn3.b"]) < 1e-10 * scale
    assert np.linalg.norm(g["block1.bn3.g"]) > 1e-4 * scale      # the scale does matter
    # and the loss itself does not move when that shift changes
    p = net.unpack(k, mods[k].astype(np.float64).copy())
    p["block1.bn3.b"] = p["block1.bn3.b"] + 0.37
    res2 = O.module_fwd_bwd(net, k, net.pack(k, p), xs[k], xs[k + 1], None, 0.7)
    assert abs(res2["loss"] - res["loss"]) < 1e-9 * abs(res["loss"])


def test_one_image_cross_entropy_gradient_stops_at_the_last_batch_norms():
    """N = 1: the adjoint of global average pooling is constant over the pixels of the only image, and the
    backward pass of a batch norm removes a per-channel constant (its statistics run over those same
    pixels).  In a post-BN block everything upstream of the last batch norms then has zero gradient."""
    cfg = small_cfg("postbn", N=1, H=16, W=16, stage_blocks=(1, 1), module_block_end=(1, 2))
    net, mods, auxs = build(cfg)
    x0 = gen.make_images(cfg).astype(np.float64)
    xs = [x0] + O.auxnet_forward(net, auxs, x0)
    res = O.module_fwd_bwd(net, 1, mods[1], xs[1], gen.make_labels(cfg), None, 1.0)
    g = net.unpack(1, res["grads"])
    scale = np.linalg.norm(res["grads"])
    for name in ("block1.conv1.w", "block1.conv2.w", "block1.sc.w", "block1.bn1.g", "block1.bn2.g", "block1.bns.g"):
        assert np.linalg.norm(g[name]) < 1e-10 * scale, name
    assert np.linalg.norm(res["dx"]) < 1e-10 * scale
    for name in ("head.fc.w", "block1.bn2.b", "block1.bns.b"):
        assert np.linalg.norm(g[name]) > 1e-3 * scale, name
