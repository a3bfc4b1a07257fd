"""GPU parity of the auxiliary-variable correction and AuxNet distillation (lp_auxnet_distill)
against the oracle: corrected variables, distillation losses, AuxNet parameter updates."""
import numpy as np
import pytest

from conftest import small_cfg
from harness import (GpuRun, NOISE_SEEDS, allowance, log_parity, noisy_bf16_store, oracle_modules, per_tensor_errors, rel_err,
                     to_dev, to_host)
from oracle import lp_oracle as O
from workloads import gen, get_config

pytestmark = pytest.mark.gpu


def distill_floors(run, xs_host, x_new, clean_grads):
    """Noise floor of every AuxNet gradient tensor of the distillation step (bf16 workloads): the largest
    change against the storage-model oracle when rounding-level noise precedes each bf16 rounding, in the
    AuxNet chain that produces the distillation input as well as in the distillation pass itself."""
    net = run.net
    floors = [dict() for _ in range(net.K - 1)]
    for seed in NOISE_SEEDS:
        net.store = noisy_bf16_store(seed)
        try:
            chain = O.auxnet_forward(net, run.auxs, run.images.astype(np.float64))
            for k in range(1, net.K):
                x_in = run.images.astype(np.float64) if k == 1 else chain[k - 2]
                res = O.auxnet_fwd_bwd(net, k - 1, run.auxs[k - 1], x_in, x_new[k - 1])
                for n, e in per_tensor_errors(net, O.LP_AUX(k - 1), res["grads"], clean_grads[k - 1]).items():
                    floors[k - 1][n] = max(floors[k - 1].get(n, 0.0), e)
        finally:
            net.store = None
    return floors


def run_case(cfg, tol, lr_lambda=0.05, lr_aux=0.01):
    run = GpuRun(cfg)
    net, lp, torch = run.net, run.lp, run.torch
    K = net.K
    bf16 = cfg["dtype"] == "bf16"
    # boundaries from the oracle's AuxNet chain under the same storage model as its distillation pass below
    # (the distillation target is x_k - lr*g_k with x_k = AuxNet_{k-1}(x_{k-1}): both must be the same x_k)
    net.store = gen.round_bf16 if bf16 else None
    ox = O.auxnet_forward(net, run.auxs, run.images, post=lambda a: gen.storage_round(a, cfg["dtype"]))
    net.store = None
    run.auxnet()                      # fills the AuxNet activations in the workspace
    run.set_boundaries(ox)            # module inputs and distillation inputs are the oracle's
    xs_host = [to_host(t) for t in run.d_x[1:]]
    run.fwd_bwd_all()
    ref = oracle_modules(run, xs_host)
    # dx_k is an argument of the call: it gets the oracle's, so that the distillation alone is compared (the
    # terminal adjoints are the library's own, held to `tol` by the step tests)
    d_dx = [None] + [to_dev(ref[k]["dx"], cfg) for k in range(1, K)]
    d_new = [torch.zeros_like(run.d_x[k]) for k in range(1, K)]
    d_loss = torch.zeros(K - 1, dtype=torch.float32, device="cuda:0")
    before = [lp.lp_get_params(run.h, lp.LP_AUX(k)).astype(np.float64) for k in range(K - 1)]
    lp.lp_auxnet_distill(run.h, run.d_images, run.d_x[1:], d_dx, lr_lambda, lr_aux, d_new, d_loss)
    assert lp.lp_last_device_status(run.h) == 0
    # oracle: same storage model as the module comparison
    net.store = gen.round_bf16 if bf16 else None
    newp, newx, losses, grads = O.auxnet_distill_step(net, run.auxs, run.images.astype(np.float64), xs_host,
                                                     [r["dx"] for r in ref[1:]], [r["seed"] for r in ref[:-1]],
                                                     lr_lambda, lr_aux)
    net.store = None
    floors = distill_floors(run, xs_host, newx, grads) if bf16 else [dict() for _ in range(K - 1)]
    got_loss = d_loss.cpu().numpy()
    bad = []
    for k in range(K - 1):
        g_gpu = lp.lp_get_grads(run.h, lp.LP_AUX(k))
        errs = per_tensor_errors(net, O.LP_AUX(k), g_gpu, grads[k])
        after = lp.lp_get_params(run.h, lp.LP_AUX(k)).astype(np.float64)
        upd = per_tensor_errors(net, O.LP_AUX(k), after - before[k], newp[k] - run.auxs[k])
        for n, e in errs.items():
            a = allowance(tol, floors[k].get(n, 0.0))
            log_parity(workload=cfg["name"] + " (distillation)", dtype=cfg["dtype"], module="aux%d" % k, tensor=n, err=e,
                       floor=floors[k].get(n, 0.0), allowed=a)
            if not e < a:
                bad.append((k, n, e, floors[k].get(n, 0.0), a))
            if not upd[n] < a + 1e-3:
                bad.append((k, n + " (update)", upd[n], floors[k].get(n, 0.0), a))
        if not rel_err(to_host(d_new[k]), newx[k]) < tol:
            bad.append((k, "x_new", rel_err(to_host(d_new[k]), newx[k])))
        if not abs(got_loss[k] - losses[k]) < 2 * tol * losses[k]:
            bad.append((k, "loss", got_loss[k], losses[k]))
    assert not bad, bad


@pytest.mark.parametrize("split", [(2, 4), (1, 3, 4)])
def test_distill_small_bf16(split):
    """K = 2 and K = 3.  With K = 3 the library's AuxNet_1 has kept activations computed from its own x_1, which
    differs from the oracle's by the rounding of a few values: the noise floor models exactly that."""
    cfg = small_cfg("preact", N=16, H=16, W=16, dtype="bf16", stage_channels=(16, 32), stage_blocks=(2, 2),
                    module_block_end=split, stem_channels=16, classes=10)
    run_case(cfg, 2e-2)


def test_distill_needs_module_passes_first():
    cfg = get_config("tiny")
    run = GpuRun(cfg)
    run.auxnet()
    with pytest.raises(run.lp.LpError) as e:
        run.lp.lp_auxnet_distill(run.h, run.d_images, run.d_x[1:], run.d_dx, 0.1, 0.1, None,
                                 run.torch.zeros(1, device="cuda:0"))
    assert e.value.status == -6


@pytest.mark.parametrize("dtype,tol", [("f32", 1e-5), ("bf16", 2e-2)])
def test_stored_auxiliary_variables_are_corrected_in_place(dtype, tol):
    """lp_aux_correct (no AuxNet): caller-held x_1..x_{K-1} (here random tensors, not AuxNet
    outputs) go through the module passes, then x_k <- x_k - lr*(dx_k - seed_{k-1}) in place;
    against the oracle's correction fed with the GPU's own dx and terminal adjoints, and against
    the x_new output of lp_auxnet_distill on the same inputs."""
    if dtype == "f32":
        cfg = small_cfg("preact", N=4, H=8, W=8, stage_channels=(8, 16), stage_blocks=(2, 2), module_block_end=(1, 3, 4))
    else:
        cfg = small_cfg("preact", N=8, H=16, W=16, dtype="bf16", stage_channels=(16, 32), stage_blocks=(2, 2),
                        module_block_end=(1, 3, 4), stem_channels=16, classes=10)
    run = GpuRun(cfg)
    net, lp, torch = run.net, run.lp, run.torch
    K = net.K
    run.auxnet()
    stored = [gen.storage_round(gen.normal(7, "stored/%d" % k, net.boundary[k], std=0.5), dtype) for k in range(1, K)]
    run.set_boundaries(stored)
    with pytest.raises(lp.LpError):                      # module passes have not run yet
        lp.lp_aux_correct(run.h, run.d_x[1:], run.d_dx, 0.1)
    run.fwd_bwd_all()
    lr = 0.1
    seeds = []
    for k in range(K - 1):
        s = torch.zeros_like(run.d_x[k + 1])
        lp.lp_get_residual(run.h, k, None, s, None)
        seeds.append(to_host(s))
    dxs = [None] + [to_host(run.d_dx[k]) for k in range(1, K)]
    want = [O.aux_correction(stored[k - 1].astype(np.float64), dxs[k], seeds[k - 1], lr)[0] for k in range(1, K)]
    d_new = [torch.zeros_like(run.d_x[k]) for k in range(1, K)]
    d_l1 = torch.zeros(K - 1, dtype=torch.float32, device="cuda:0")
    lp.lp_auxnet_distill(run.h, run.d_images, run.d_x[1:], run.d_dx, lr, 0.0, d_new, d_l1)
    d_l2 = torch.zeros(K - 1, dtype=torch.float32, device="cuda:0")
    lp.lp_aux_correct(run.h, run.d_x[1:], run.d_dx, lr, d_l2)
    assert lp.lp_last_device_status(run.h) == 0
    np.testing.assert_allclose(d_l2.cpu().numpy(), d_l1.cpu().numpy(), rtol=1e-5)
    for k in range(1, K):
        got = to_host(run.d_x[k])
        np.testing.assert_array_equal(got, to_host(d_new[k - 1]))
        assert rel_err(got, want[k - 1]) < tol
        g = dxs[k].astype(np.float64) - seeds[k - 1]
        assert abs(float(d_l2[k - 1]) - lr * lr * float((g * g).sum())) < 1e-4 * lr * lr * float((g * g).sum()) + 1e-12
