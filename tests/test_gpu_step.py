"""GPU parity of the whole layer-parallel step against the oracle, through the C ABI.

Tolerances (relative L2 error per tensor): 1e-4 on the fp32 path, 2e-2 on the bf16 path, for
losses, parameter gradients, input gradients, AuxNet outputs and updated parameters.
"""
import numpy as np
import pytest

from conftest import small_cfg
from harness import GpuRun, allowance, log_parity, noise_floors, oracle_modules, per_tensor_errors, rel_err, to_host
from oracle import lp_oracle as O
from workloads import gen, get_config, scaled

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}


def check_modules(run, grads, ref, tol, floors=None, dx_from=1):
    """Per-tensor relative L2 errors of parameter gradients, input gradients and losses.

    fp32: every tensor within `tol`.  bf16: within harness.allowance(tol, floor) = max(tol, min(2 x floor, 0.20)),
    the floor being the largest change of that tensor between the storage-model oracle and runs of it that differ
    by 1e-7 relative noise before each bf16 rounding (harness.noise_floors); losses always within `tol`.
    Every comparison is also written to the parity log (harness.log_parity)."""
    net = run.net
    loss = run.d_loss.cpu().numpy()
    allow, bad = [], []

    def check(k, tensor, err, floor, allowed):
        log_parity(workload=run.cfg["name"], dtype=run.cfg["dtype"], module=k, tensor=tensor, err=float(err),
                   floor=float(floor), allowed=float(allowed))
        if not err < allowed:
            bad.append((k, tensor, float(err), float(floor), float(allowed)))

    for k in range(net.K):
        errs = per_tensor_errors(net, k, grads[k], ref[k]["grads"])
        fl = floors[k]["grads"] if floors else {}
        allow.append({n: allowance(tol, fl.get(n, 0.0)) for n in errs})
        blob = float(np.linalg.norm(ref[k]["grads"]))
        off = 0
        for name, _, shape in net.param_layout(k):
            n_el = int(np.prod(shape))
            sl = slice(off, off + n_el)
            off += n_el
            if fl.get(name, 0.0) >= 0.5:
                # Undetermined tensor: the oracle's own runs under rounding noise differ from one another by
                # more than half the tensor's norm (a gradient that vanishes in exact arithmetic and is pure
                # rounding residue with bf16 storage).  It has no scale of its own; it is held, in absolute
                # terms, to `tol` of the norm of the module's whole gradient.
                e_abs = float(np.linalg.norm(np.asarray(grads[k][sl], dtype=np.float64) - ref[k]["grads"][sl])) / blob
                allow[k][name] = tol
                check(k, name + " (undetermined; |diff| / |whole gradient|)", e_abs, fl[name], tol)
            else:
                check(k, name, errs[name], fl.get(name, 0.0), allow[k][name])
        whole_floor = floors[k]["whole"] if floors else 0.0
        check(k, "(whole gradient)", rel_err(grads[k], ref[k]["grads"]), whole_floor, allowance(tol, whole_floor))
        check(k, "(loss)", abs(loss[k, 0] - ref[k]["loss"]) / max(abs(ref[k]["loss"]), 1e-30), 0.0, tol)
        if k < net.K - 1:
            check(k, "(residual norm)", abs(loss[k, 1] - ref[k]["rnorm2"]) / ref[k]["rnorm2"], 0.0, tol)
        if k >= dx_from:
            f = floors[k]["dx"] if floors else 0.0
            check(k, "(dx)", rel_err(to_host(run.d_dx[k]), ref[k]["dx"]), f, allowance(tol, f))
    assert not bad, bad          # (module, tensor, error, floor, allowed)
    return allow


def full_step_parity(cfg, conv_impl=0, grouped=True, steps=1):
    run = GpuRun(cfg, conv_impl=conv_impl)
    net, tol = run.net, TOL[cfg["dtype"]]
    # AuxNet chain: GPU against oracle (the oracle feeds each AuxNet the storage-rounded tensor)
    post = (lambda a: gen.storage_round(a, cfg["dtype"]))
    ox = O.auxnet_forward(net, run.auxs, run.images, post=post)
    gx = run.auxnet()
    for k in range(net.K - 1):
        assert rel_err(gx[k], ox[k]) < tol, ("auxnet", k, rel_err(gx[k], ox[k]))
    # module inputs come from the oracle, never from the CUDA path
    run.set_boundaries(ox)
    xs_host = [to_host(t) for t in run.d_x[1:]]
    params = [m.astype(np.float64) for m in run.mods]
    kappas = [k.astype(np.float64) for k in run.kappa] if run.use_kappa else None
    lr = None
    for step in range(steps):
        grads = run.fwd_bwd_all(grouped=grouped)
        ref = oracle_modules(run, xs_host, kappas=kappas, params=params)
        floors = noise_floors(run, xs_host, ref, kappas=kappas, params=params) if cfg["dtype"] == "bf16" else None
        allow = check_modules(run, grads, ref, tol, floors)
        if cfg["dtype"] == "bf16" and step == 0:
            # against exact arithmetic: losses and residual norms within the same tolerance
            exact = oracle_modules(run, xs_host, kappas=kappas, params=params, exact=True)
            loss = run.d_loss.cpu().numpy()
            for k in range(net.K):
                assert abs(loss[k, 0] - exact[k]["loss"]) < tol * abs(exact[k]["loss"]), (k, "exact loss")
        for k in range(net.K - 1):
            r = run.torch.zeros_like(run.d_x[k + 1])
            s = run.torch.zeros_like(run.d_x[k + 1])
            run.lp.lp_get_residual(run.h, k, r, s)
            assert rel_err(to_host(r), ref[k]["r"]) < tol
            assert rel_err(to_host(s), ref[k]["seed"]) < tol
        if lr is None:
            # the penalty is a plain sum over the boundary tensor, so gradients are large: pick the
            # learning rate (from the oracle's gradients) that moves the parameters by about 0.02
            lr = 0.02 / max(float(np.abs(ref[k]["grads"]).max()) for k in range(net.K))
        run.cfg["lr"] = lr
        before = [run.lp.lp_get_params(run.h, k).astype(np.float64) for k in range(net.K)]
        run.step()
        new_params = [O.sgd_update(params[k], ref[k]["grads"], lr)[0] for k in range(net.K)]
        for k in range(net.K):
            got = run.lp.lp_get_params(run.h, k).astype(np.float64)
            errs = per_tensor_errors(net, k, got, new_params[k])
            assert max(errs.values()) < tol, (k, errs)
            # the update itself, wherever it is large enough to be resolved in the fp32 master copy
            off = 0
            for name, _, shape in net.param_layout(k):
                n = int(np.prod(shape))
                sl = slice(off, off + n)
                off += n
                d_ref = new_params[k][sl] - params[k][sl]
                if np.linalg.norm(d_ref) > 2e-3 * np.linalg.norm(params[k][sl]):
                    assert rel_err(got[sl] - before[k][sl], d_ref) < allow[k][name] + 1e-3, (k, name)
        params = new_params
        if kappas is not None:
            kappas = [O.kappa_update(kappas[k], ref[k]["r"], cfg["rho"]) for k in range(net.K - 1)]
            for k in range(net.K - 1):
                assert rel_err(to_host(run.d_kappa[k]), kappas[k]) < tol
        # The oracle continues from its own updated parameters and multipliers.  On the bf16 path
        # the GPU's second step is started from the oracle's state as well: its own fp32 masters
        # differ from the oracle's by the (already checked) gradient error times the learning
        # rate, which is enough to flip a few ReLU masks and would be counted twice.
        if cfg["dtype"] == "bf16" and step + 1 < steps:
            for k in range(net.K):
                run.lp.lp_set_params(run.h, k, params[k].astype(np.float32))
                params[k] = params[k].astype(np.float32).astype(np.float64)
            if kappas is not None:
                for k in range(net.K - 1):
                    kq = gen.round_bf16(kappas[k])
                    run.d_kappa[k].copy_(run.torch.from_numpy(kq).to("cuda:0").to(run.torch.bfloat16))
                    kappas[k] = kq.astype(np.float64)
    return run


def test_tiny_fp32_step_two_steps():
    full_step_parity(get_config("tiny"), steps=2)


def test_tiny_fp32_per_module_calls_and_penalty():
    cfg = get_config("tiny")
    cfg["loss"] = "penalty"
    full_step_parity(cfg, grouped=False)


@pytest.mark.parametrize("kind,stem", [("postbn", "conv3x3"), ("preact", "conv3x3"), ("postbn", "conv7x7s2_maxpool")])
def test_small_fp32_block_kinds(kind, stem):
    if stem == "conv3x3":
        cfg = small_cfg(kind, N=4, H=8, W=8)
    else:
        cfg = small_cfg(kind, stem=stem, N=3, H=32, W=32, stage_channels=(8, 16), stage_stride=(1, 2))
    full_step_parity(cfg, steps=1)


# CUDA cores; tensor cores; direct / staged epilogue everywhere; batch-norm backward sums in the conv epilogue
@pytest.mark.parametrize("impl", [1, 0, 256, 512, 2048])
@pytest.mark.parametrize("kind", ["postbn", "preact"])
def test_small_bf16_block_kinds(kind, impl):
    cfg = small_cfg(kind, N=8, H=16, W=16, dtype="bf16", stage_channels=(16, 32), stage_blocks=(2, 2),
                    module_block_end=(1, 3, 4), stem_channels=16, classes=10)
    full_step_parity(cfg, conv_impl=impl, steps=2)


@pytest.mark.parametrize("kind", ["postbn", "preact", "bottleneck"])
def test_bn_backward_sums_in_the_conv_epilogue_equal_the_separate_kernel(kind):
    """The reduction pass of a batch-norm backward taken by the epilogue of the input-gradient convolution
    (LP_CONV_BN_REDUCE_IN_EPILOGUE) against the same pass as its own kernel (default): the same bf16 values are
    summed, only the order of the fp32 additions differs, so the gradients agree far inside the parity
    tolerance; the launch count shows that the kernels are really gone."""
    import paper_2112_05387_b200 as lp
    cfg = small_cfg(kind, N=8, H=16, W=16, dtype="bf16", stage_channels=(16, 32) if kind != "bottleneck" else (64, 128),
                    stage_blocks=(2, 2), module_block_end=(1, 3, 4), stem_channels=16, classes=10)
    out = {}
    for impl in (lp.LP_CONV_BN_REDUCE_IN_EPILOGUE, 0):
        run = GpuRun(cfg, conv_impl=impl)
        run.auxnet()
        run.lp.lp_launch_count(run.h, reset=True)
        grads = run.fwd_bwd_all()
        out[impl] = (grads, [to_host(t) for t in run.d_dx[1:]], run.d_loss.cpu().numpy().copy(),
                     run.lp.lp_last_device_status(run.h), run.lp.lp_launch_count(run.h))
        run.lp.lp_destroy(run.h)
    (g0, dx0, l0, s0, n0), (g1, dx1, l1, s1, n1) = out[lp.LP_CONV_BN_REDUCE_IN_EPILOGUE], out[0]
    assert s0 == 0 and s1 == 0
    assert n0 <= n1 - 4, (n0, n1)                         # at least one reduction kernel per block is gone
    np.testing.assert_array_equal(l0, l1)                 # the forward pass is untouched
    for k in range(len(g0)):
        assert rel_err(g0[k], g1[k]) < 2e-3, k
    for a, b in zip(dx0, dx1):
        assert rel_err(a, b) < 2e-3


def test_weight_gradients_on_their_own_stream_equal_those_in_the_chain():
    """A module's weight gradients run on a second stream by default and inside the module's stream with
    LP_CONV_WGRAD_IN_CHAIN: the same kernels on the same operands, so losses are identical and gradients agree
    to the order of the fp32 reductions; run twice to show that nothing races between the two streams."""
    import paper_2112_05387_b200 as lp
    cfg = small_cfg("postbn", N=8, H=16, W=16, dtype="bf16", stage_channels=(16, 32), stage_blocks=(2, 2),
                    module_block_end=(1, 3, 4), stem_channels=16, classes=10)
    out = []
    for impl in (0, 0, lp.LP_CONV_WGRAD_IN_CHAIN):
        run = GpuRun(cfg, conv_impl=impl)
        run.auxnet()
        grads = run.fwd_bwd_all()
        out.append((grads, run.d_loss.cpu().numpy().copy(), run.lp.lp_last_device_status(run.h)))
        run.lp.lp_destroy(run.h)
    for g, l, st in out:
        assert st == 0
        np.testing.assert_array_equal(l, out[0][1])
        for k in range(len(g)):
            assert rel_err(g[k], out[0][0][k]) < 1e-5, k


def flat_module_parity(cfg, conv_impl, tol_grad):
    """Module passes of a bf16 network against the storage-model oracle with ONE tolerance for every
    gradient tensor and dx, no noise floor: for networks shallow enough that rounding-level differences
    do not reach a mask."""
    run = GpuRun(cfg, conv_impl=conv_impl)
    net = run.net
    ox = O.auxnet_forward(net, run.auxs, run.images, post=lambda a: gen.storage_round(a, cfg["dtype"]))
    run.set_boundaries(ox)
    xs_host = [to_host(t) for t in run.d_x[1:]]
    grads = run.fwd_bwd_all()
    ref = oracle_modules(run, xs_host)
    flat = [dict(grads={}, whole=0.0, dx=0.0) for _ in range(net.K)]     # floor 0: the allowance is the tolerance
    check_modules(run, grads, ref, tol_grad, flat)


@pytest.mark.parametrize("kind,tol", [("postbn", 5e-3), ("preact", 1.5e-2)])
def test_bf16_backward_arithmetic_on_cuda_cores_depth_four(kind, tol):
    """CUDA-core convolutions read the same bf16 operand values as the oracle's storage model and accumulate
    in fp32: with nothing but the accumulation differing, every gradient tensor and dx of a four-block network
    stays within a flat 5e-3 (post-BN blocks; seen 3.1e-3) or 1.5e-2 (pre-activation blocks; seen 1.0e-2 in the
    two-block module, whose first batch norm works on the module input).  This pins the backward arithmetic
    of the bf16 path (batch-norm backward, masks recomputed from stored values, residual fan-in, storage
    points) apart from the tensor-core kernels."""
    import paper_2112_05387_b200 as lp
    cfg = small_cfg(kind, N=8, H=16, W=16, dtype="bf16", stage_channels=(16, 32), stage_blocks=(2, 2),
                    module_block_end=(1, 3, 4), stem_channels=16, classes=10)
    flat_module_parity(cfg, lp.LP_CONV_IMPL_SIMT, tol)


@pytest.mark.parametrize("kind", ["postbn", "preact", "bottleneck"])
def test_bf16_shallow_network_on_tensor_cores_flat_tolerance(kind):
    """One block per module on the tensor-core kernels: 2e-2 for every tensor, no allowance for noise."""
    ch = (64, 128) if kind == "bottleneck" else (16, 32)
    cfg = small_cfg(kind, N=8, H=16, W=16, dtype="bf16", stage_channels=ch, stage_blocks=(1, 1),
                    module_block_end=(1, 2), stem_channels=16, classes=10)
    flat_module_parity(cfg, 0, 2e-2)


@pytest.mark.parametrize("loss", ["penalty", "al"])
def test_local_loss_sums_with_160_channels_match_a_host_sum(loss):
    """Boundary tensors of 160 bf16 channels (the wide-ResNet width: the loss kernel then runs blocks of
    240 threads, whose last warp is partial) on a tensor large enough that dozens of blocks contribute:
    sum r^2 and sum kappa*r as returned by the call against sums of the stored residual taken on the host."""
    cfg = small_cfg("preact", N=8, H=16, W=16, dtype="bf16", stage_channels=(160, 320), stage_blocks=(1, 1),
                    module_block_end=(1, 2), stem_channels=16, classes=10, aux_width_div=4)
    cfg["loss"] = loss
    run = GpuRun(cfg)
    run.auxnet()
    run.fwd_bwd_all()
    r = run.torch.zeros_like(run.d_x[1])
    run.lp.lp_get_residual(run.h, 0, r, None)
    r = to_host(r)
    assert r.shape[-1] == 160 and r.size >= 40 * 240 * 8
    loss_dev = run.d_loss.cpu().numpy()
    rr = float((r * r).sum())
    kr = float((to_host(run.d_kappa[0]) * r).sum()) if loss == "al" else 0.0
    assert abs(loss_dev[0, 1] - rr) < 2e-3 * rr                      # r is read back in bf16
    want = 0.5 * cfg["rho"] * rr + kr
    assert abs(loss_dev[0, 0] - want) < 2e-3 * abs(want)


@pytest.mark.parametrize("impl", [0, 64])
def test_bf16_stem_7x7_stride_2_on_tensor_cores(impl):
    """The ImageNet-shaped stem (7x7 / stride 2 / pad 3, 3 input channels, max-pool) of a bf16 network runs on
    the tensor cores by space-to-depth (a 4x4 stride-1 convolution over 2x2 pixel blocks): module 0's
    gradients, stem weights included, at a flat 2e-2 against the storage-model oracle.  impl = 64 keeps the
    weight gradients on the CUDA cores (the stem then takes the plain kernels): same bound."""
    cfg = small_cfg("postbn", stem="conv7x7s2_maxpool", N=6, H=48, W=40, dtype="bf16", stem_channels=16,
                    stage_channels=(16, 32), stage_blocks=(1, 1), module_block_end=(1, 2), classes=10)
    flat_module_parity(cfg, impl, 2e-2)


def test_resnet56_reduced_batch_bf16():
    full_step_parity(scaled("resnet56", N=16), steps=1)


def test_resnet110_reduced_batch_bf16_two_steps():
    full_step_parity(scaled("resnet110", N=8), steps=2)


def test_wrn28_10_reduced_batch_bf16():
    full_step_parity(scaled("wrn28_10", N=6), steps=1)


def test_wrn28_10_reduced_batch_bf16_on_cta_pairs():
    """LP_CONV_TWO_CTA: the 3x3 stride-1 layers (forward and input gradient, with and without a residual operand,
    with statistics) on pairs of CTAs give the same step."""
    import paper_2112_05387_b200 as lp
    full_step_parity(scaled("wrn28_10", N=6), conv_impl=lp.LP_CONV_TWO_CTA, steps=1)


def test_wrn28_10_loss_in_the_last_convolutions_epilogue():
    """LP_CONV_LOSS_IN_EPILOGUE: residual, loss sums and terminal adjoint taken by the epilogue of each
    interior module's last convolution give the same step as the separate pass (penalty and AL)."""
    import paper_2112_05387_b200 as lp
    full_step_parity(scaled("wrn28_10", N=6), conv_impl=lp.LP_CONV_LOSS_IN_EPILOGUE, steps=1)
    cfg = scaled("wrn28_10", N=4)
    cfg["loss"] = "al"
    cfg["kappa_std"] = 0.1
    full_step_parity(cfg, conv_impl=lp.LP_CONV_LOSS_IN_EPILOGUE, steps=1)


def test_bottleneck_blocks_fp32():
    """1x1 - 3x3 - 1x1 blocks: identity and projection shortcuts, a stride-2 block, a module boundary inside a stage."""
    cfg = small_cfg("bottleneck", N=4, H=8, W=8, stage_channels=(16, 32), stage_blocks=(2, 2), module_block_end=(1, 3, 4),
                    stem_channels=16)
    full_step_parity(cfg, steps=2)


def test_bottleneck_blocks_bf16_tensor_cores():
    cfg = small_cfg("bottleneck", N=8, H=16, W=16, dtype="bf16", stage_channels=(64, 128), stage_blocks=(2, 2),
                    module_block_end=(1, 3, 4), stem_channels=16, classes=10)
    full_step_parity(cfg, steps=1)


def test_resnet50_reduced_bf16():
    full_step_parity(scaled("resnet50", N=2, H=64, W=64), steps=1)


@pytest.mark.parametrize("kind", ["postbn", "preact", "bottleneck"])
def test_degenerate_split_one_module_is_ordinary_backpropagation(kind):
    """K = 1: no auxiliary variable, no AuxNet, no interior loss; the step is plain BP of the cross-entropy."""
    ch = (16, 32) if kind == "bottleneck" else (8, 16)
    cfg = small_cfg(kind, N=4, H=8, W=8, stage_channels=ch, stage_blocks=(1, 1), module_block_end=(2,),
                    stem_channels=ch[0])
    run = full_step_parity(cfg, steps=2)
    assert run.net.K == 1 and run.lp.lp_workspace_bytes(run.desc) > 0


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_batch_of_two_images(dtype):
    """N = 2, the smallest batch whose last-module gradients do not vanish identically (with one image the
    adjoint of the pooled head is constant over the pixels and the last batch norms remove it: an oracle
    pin); tiles are mostly ragged."""
    kw = dict(stem_channels=16, stage_channels=(16, 32), classes=10) if dtype == "bf16" else {}
    cfg = small_cfg("postbn", N=2, H=16, W=16, dtype=dtype, stage_blocks=(1, 1), module_block_end=(1, 2), **kw)
    full_step_parity(cfg, steps=1)


def test_batch_of_one_image_runs_and_matches_in_the_forward_quantities():
    cfg = small_cfg("postbn", N=1, H=16, W=16, stage_blocks=(1, 1), module_block_end=(1, 2))
    run = GpuRun(cfg)
    post = (lambda a: gen.storage_round(a, cfg["dtype"]))
    ox = O.auxnet_forward(run.net, run.auxs, run.images, post=post)
    gx = run.auxnet()
    assert rel_err(gx[0], ox[0]) < 1e-4
    run.set_boundaries(ox)
    grads = run.fwd_bwd_all()
    ref = oracle_modules(run, [to_host(t) for t in run.d_x[1:]])
    loss = run.d_loss.cpu().numpy()
    for k in range(2):
        assert abs(loss[k, 0] - ref[k]["loss"]) < 1e-4 * abs(ref[k]["loss"])
    errs = per_tensor_errors(run.net, 0, grads[0], ref[0]["grads"])      # the interior module is not degenerate
    assert max(errs.values()) < 1e-4, errs
    # last module: only the head and the shifts of the last batch norms receive a gradient
    g = run.net.unpack(1, grads[1])
    r = run.net.unpack(1, ref[1]["grads"])
    for name in ("head.fc.w", "head.fc.b", "block1.bn2.b", "block1.bns.b"):
        assert rel_err(g[name], r[name]) < 1e-4, name
    scale = np.linalg.norm(ref[1]["grads"])
    for name in ("block1.conv1.w", "block1.conv2.w", "block1.sc.w", "block1.bn2.g"):
        assert np.linalg.norm(r[name]) < 1e-9 * scale and np.linalg.norm(g[name]) < 1e-5 * scale, name


def test_every_block_its_own_module():
    """The finest split: K = number of blocks (module boundaries at a stride-2 block's entry included)."""
    cfg = small_cfg("preact", N=4, H=16, W=16, stage_channels=(8, 16, 32), stage_blocks=(2, 2, 2), stage_stride=(1, 2, 2),
                    module_block_end=(1, 2, 3, 4, 5, 6))
    run = full_step_parity(cfg, steps=1)
    assert run.net.K == 6


def test_resnet34_reduced_bf16():
    full_step_parity(scaled("resnet34", N=2, H=64, W=64), steps=1)


def test_serial_forward_matches_oracle_and_serial_backprop_is_bp():
    """Layer-serial comparator: x_{k+1} := F_k(x_k) reproduces the undecomposed network, and
    back-propagating the cross-entropy through all modules gives the ordinary BP gradients."""
    cfg = small_cfg("preact", N=4, H=8, W=8, stage_channels=(8, 16), stage_blocks=(2, 2), module_block_end=(1, 3, 4))
    run = GpuRun(cfg)
    torch = run.torch
    logits = torch.zeros(cfg["N"], cfg["num_classes"], dtype=torch.float32, device="cuda:0")
    run.lp.lp_forward_serial(run.h, run.d_images, logits)
    assert run.lp.lp_last_device_status(run.h) == 0
    ref = O.forward_serial(run.net, run.mods, run.images)
    assert rel_err(logits.cpu().numpy(), ref) < 1e-4
    loss = torch.zeros(2, dtype=torch.float32, device="cuda:0")
    run.lp.lp_serial_fwd_bwd(run.h, run.d_images, run.d_labels, loss)
    assert run.lp.lp_last_device_status(run.h) == 0
    # oracle BP: chain the modules, seed each with the next module's input gradient
    net = run.net
    xs = [run.images.astype(np.float64)]
    for k in range(net.K - 1):
        xs.append(O.module_forward(net, k, net.unpack(k, run.mods[k]), xs[k]))
    res = O.module_fwd_bwd(net, net.K - 1, run.mods[-1], xs[-1], run.labels, None, 1.0)
    assert abs(loss[0].item() - res["loss"]) < 1e-4 * abs(res["loss"])
    errs = per_tensor_errors(net, net.K - 1, run.lp.lp_get_grads(run.h, net.K - 1), res["grads"])
    assert max(errs.values()) < 1e-4, errs
    # module K-2 receives dx of module K-1 as terminal adjoint: penalty with rho = 0 and kappa = dx
    d = res["dx"]
    for k in range(net.K - 2, -1, -1):
        r2 = O.module_fwd_bwd(net, k, run.mods[k], xs[k], xs[k + 1], d, 0.0)
        errs = per_tensor_errors(net, k, run.lp.lp_get_grads(run.h, k), r2["grads"])
        assert max(errs.values()) < 2e-4, (k, errs)
        d = r2["dx"]


@pytest.mark.parametrize("which", ["tiny", "bf16-preact", "bf16-postbn"])
def test_fused_step_equals_the_three_separate_calls(which):
    """lp_layer_parallel_step (AuxNet stream, per-module start / loss / update events) computes what
    lp_auxnet_forward + lp_modules_fwd_bwd_all + lp_step compute: same boundaries, losses, gradients,
    updated parameters and multipliers (only the order of fp32 atomic sums differs)."""
    if which == "tiny":
        cfg, tol = get_config("tiny"), 1e-5
    else:
        cfg = small_cfg(which.split("-")[1], N=8, H=16, W=16, dtype="bf16", stage_channels=(16, 32), stage_blocks=(2, 2),
                        module_block_end=(1, 3, 4), stem_channels=16, classes=10)
        tol = 2e-2
    a, b = GpuRun(cfg), GpuRun(cfg)
    K, lp = a.net.K, a.lp
    lr, c = 1e-4, cfg["rho"]
    a.cfg["lr"] = lr
    a.auxnet()
    ga = a.fwd_bwd_all()
    a.step(kappa_step=c)
    lp.lp_layer_parallel_step(b.h, b.d_images, b.d_x[1:], b.d_labels, b.d_kappa if b.use_kappa else None, cfg["rho"],
                              b.d_loss, b.d_dx, lr, 0.0, 0.0, c)
    assert lp.lp_last_device_status(b.h) == 0
    for k in range(1, K):
        assert rel_err(to_host(b.d_x[k]), to_host(a.d_x[k])) < tol
        assert rel_err(to_host(b.d_dx[k]), to_host(a.d_dx[k])) < tol
    np.testing.assert_allclose(b.d_loss.cpu().numpy(), a.d_loss.cpu().numpy(), rtol=max(tol, 1e-5))
    for k in range(K):
        assert rel_err(lp.lp_get_grads(b.h, k), ga[k]) < tol
        assert rel_err(lp.lp_get_params(b.h, k), lp.lp_get_params(a.h, k)) < tol
    if a.use_kappa:
        for k in range(K - 1):
            assert rel_err(to_host(b.d_kappa[k]), to_host(a.d_kappa[k])) < tol


def test_timeline_records_every_operation_of_a_step():
    """lp_timeline: one record per operation and phase, ordered in time within a module, and a
    step run with the time line enabled gives the same losses as one without."""
    cfg = get_config("tiny")
    run = GpuRun(cfg)
    lp, h, K = run.lp, run.h, run.net.K
    lam = run.d_kappa if run.use_kappa else None

    def step():
        lp.lp_layer_parallel_step(h, run.d_images, run.d_x[1:], run.d_labels, lam, cfg["rho"], run.d_loss, run.d_dx,
                                  0.0, 0.0, 0.0, 0.0)
        assert lp.lp_last_device_status(h) == 0
        return to_host(run.d_loss).copy()

    ref = step()
    assert lp.lp_timeline(h, True, read=False) == []
    got = step()
    recs = lp.lp_timeline(h, False)
    np.testing.assert_array_equal(got, ref)
    assert lp.lp_timeline(h, False) == []          # reading drops the records
    phases = {r["phase"] for r in recs}
    assert {"aux_forward", "forward", "backward", "update"} <= phases
    for k in range(K):
        mine = [r for r in recs if r["plan"] == k]
        assert sum(r["op"] == "update" for r in mine) == 1
        assert sum(r["op"] == "out_loss" for r in mine) == (1 if k < K - 1 else 0)
        assert sum(r["op"] == "head_fwd" for r in mine) == (1 if k == K - 1 else 0)
        n_fwd = sum(r["op"] == "conv_fwd" for r in mine)
        assert n_fwd == sum(r["op"] == "conv_wgrad" for r in mine) and n_fwd >= 2
        # operations of one module run on one stream, in the order they were issued
        for a, b in zip(mine, mine[1:]):
            assert a["start_ms"] <= a["end_ms"] <= b["start_ms"] + 1e-3
        order = [r["phase"] for r in mine]
        assert order == sorted(order, key=["forward", "backward", "update"].index)
    assert all(r["plan"] >= 256 for r in recs if r["phase"] == "aux_forward")
    assert min(r["start_ms"] for r in recs) == 0.0
    # a graph cannot hold events that are read back: recording is refused while the time line is on
    lp.lp_timeline(h, True, read=False)
    with pytest.raises(lp.LpError):
        lp.lp_graph_begin(h, None)
    lp.lp_timeline(h, False, read=False)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_update_with_momentum_and_weight_decay(dtype):
    """lp_step with heavy-ball momentum and weight decay, two steps from the same gradients, against
    the oracle's update (the velocity starts at zero).  fp32 nets take the plain update kernel; bf16
    nets the pass that also refreshes the packed bf16 weights, so the second forward must see them."""
    if dtype == "f32":
        cfg = get_config("tiny")
    else:
        cfg = small_cfg("preact", N=8, H=16, W=16, dtype="bf16", stage_channels=(16, 32), stage_blocks=(1, 1),
                        module_block_end=(1, 2), stem_channels=16, classes=10)
    run = GpuRun(cfg)
    lp, h, K = run.lp, run.h, run.net.K
    run.auxnet()
    grads = run.fwd_bwd_all()
    scale = max(np.abs(g).max() for g in grads)
    lr, mom, wd = 0.05 / scale, 0.9, 0.01
    p0 = [lp.lp_get_params(h, k) for k in range(K)]
    lp.lp_step(h, lr, mom, wd, 0.0, None)
    p1 = [lp.lp_get_params(h, k) for k in range(K)]
    vel = []
    for k in range(K):
        want, v = O.sgd_update(p0[k], grads[k], lr, momentum=mom, weight_decay=wd)
        vel.append(v)
        np.testing.assert_allclose(p1[k], want, rtol=2e-6, atol=1e-7)
    # second step: same inputs, new parameters; the oracle update uses the GPU's own new gradients
    loss_before = to_host(run.d_loss).copy()
    grads2 = run.fwd_bwd_all()
    assert not np.array_equal(to_host(run.d_loss), loss_before)   # the forward used the updated weights
    lp.lp_step(h, lr, mom, wd, 0.0, None)
    for k in range(K):
        want, _ = O.sgd_update(p1[k], grads2[k], lr, momentum=mom, weight_decay=wd, velocity=vel[k])
        np.testing.assert_allclose(lp.lp_get_params(h, k), want, rtol=2e-6, atol=1e-7)


def test_speedup_accounting_on_the_tiny_workload():
    """The speed-up accounting (Section 4.3) runs end to end: K = 1 has no auxiliary phases and the
    model ratio 1; K = 2 has all five phases and a model ratio between 1 and K."""
    from paper_2112_05387_b200 import speedup_accounting as sa
    one = sa.measure("tiny", 1, reps=3)
    two = sa.measure("tiny", 2, reps=3)
    assert one["module_block_end"] == [2] and two["module_block_end"] == [1, 2]
    p1, p2 = one["phases_ms"], two["phases_ms"]
    assert p1["t_psi"] == p1["t_f_lambda"] == p1["t_b_lambda"] == 0.0 and one["rho_model_K_devices"] == 1.0
    assert all(v > 0 for v in p2.values())
    assert 1.0 < two["rho_model_K_devices"] < 2.0
    for r in (one, two):
        assert all(v > 0 for v in r["step_ms"].values())
        assert r["rho_measured_one_gpu"] == pytest.approx(r["step_ms"]["layer_serial"] / r["step_ms"]["layer_parallel"])


def test_argument_errors_are_reported_on_the_host():
    cfg = get_config("tiny")
    run = GpuRun(cfg)
    lp = run.lp
    with pytest.raises(lp.LpError) as e:
        lp.lp_module_fwd_bwd(run.h, 5, run.d_x[0], run.d_x[1], None, 1.0, run.d_loss[0], None)
    assert e.value.status == -3
    with pytest.raises(lp.LpError) as e:
        lp.lp_module_fwd_bwd(run.h, 0, None, run.d_x[1], None, 1.0, run.d_loss[0], None)
    assert e.value.status == -1
    with pytest.raises(lp.LpError) as e:
        lp.lp_module_fwd_bwd(run.h, 0, run.d_x[0].data_ptr() + 4, run.d_x[1], None, 1.0, run.d_loss[0], None)
    assert e.value.status == -4
    with pytest.raises(lp.LpError) as e:
        lp.lp_step(run.h, 0.1)
    assert e.value.status == -6
    with pytest.raises(lp.LpError) as e:
        lp.lp_set_params(run.h, 0, np.zeros(3, dtype=np.float32))
    assert e.value.status == -9
    assert lp.lp_last_device_status(run.h) == 0


def test_a_device_wait_that_runs_out_is_reported_and_the_handle_stays_usable():
    """The bounded device-side wait behind LP_ERR_DEVICE_TIMEOUT: a thread waits 0.5 ms on a barrier that
    nothing signals, gives up, records it and returns.  The status call reports the time-out once, and an
    ordinary step afterwards passes and matches the step before it."""
    cfg = get_config("tiny")
    run = GpuRun(cfg)
    lp = run.lp
    run.auxnet()
    g0 = run.fwd_bwd_all()
    waited = lp.lp_selftest_bounded_wait(run.h, 0.5)
    assert 0.4 < waited < 50.0, waited                 # it did wait about the limit, and it did stop
    assert lp.lp_last_device_status(run.h) == -7 and "timed out" in lp.lp_status_string(-7)
    assert lp.lp_last_device_status(run.h) == 0        # reported once, then cleared
    g1 = run.fwd_bwd_all()                             # asserts a clean device status itself
    for a, b in zip(g0, g1):
        assert rel_err(a, b) < 1e-5                    # fp32 atomic sums: the order differs between runs
    with pytest.raises(lp.LpError):
        lp.lp_selftest_bounded_wait(run.h, 1e6)        # limits beyond 100 ms are refused


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_parameters_saved_and_restored_give_the_same_step(dtype):
    """Checkpoint round trip: lp_get_params -> one step -> lp_set_params of the saved blobs -> the same
    step again gives the same losses, gradients and updated parameters (the bf16 operand copies of the
    weights are rebuilt by lp_set_params)."""
    if dtype == "f32":
        cfg = get_config("tiny")
    else:
        cfg = small_cfg("preact", N=8, H=16, W=16, dtype="bf16", stage_channels=(16, 32), stage_blocks=(1, 1),
                        module_block_end=(1, 2), stem_channels=16, classes=10)
    run = GpuRun(cfg)
    lp, h, K = run.lp, run.h, run.net.K
    run.auxnet()
    kappa0 = [t.clone() for t in run.d_kappa]
    saved = [lp.lp_get_params(h, k) for k in range(K)]
    saved_aux = [lp.lp_get_params(h, lp.LP_AUX(k)) for k in range(K - 1)]
    run.cfg["lr"] = 1e-3

    def one_step():
        grads = run.fwd_bwd_all()
        loss = to_host(run.d_loss).copy()
        run.step()
        return grads, loss, [lp.lp_get_params(h, k) for k in range(K)], [to_host(t) for t in run.d_kappa]

    g1, l1, p1, k1 = one_step()
    assert any(not np.array_equal(a, b) for a, b in zip(p1, saved))      # the step did move the parameters
    for k in range(K):
        lp.lp_set_params(h, k, saved[k])
    for k in range(K - 1):
        lp.lp_set_params(h, lp.LP_AUX(k), saved_aux[k])
    for t, t0 in zip(run.d_kappa, kappa0):                               # multipliers are the caller's state
        t.copy_(t0)
    for k in range(K):
        np.testing.assert_array_equal(lp.lp_get_params(h, k), saved[k])
    g2, l2, p2, k2 = one_step()
    rtol = 1e-5 if dtype == "f32" else 2e-3      # weight gradients are summed with atomics: order differs
    np.testing.assert_allclose(l2, l1, rtol=rtol)
    for k in range(K):
        assert rel_err(g2[k], g1[k]) < rtol
        assert rel_err(p2[k], p1[k]) < rtol
    for a, b in zip(k2, k1):
        assert rel_err(a, b) < rtol
