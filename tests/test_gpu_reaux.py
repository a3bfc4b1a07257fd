"""GPU parity of the recursive auxiliary-variable networks (descriptor aux_recursive = 1; Eq. ReAuxNet-FP,
Eq. ReAuxNet-Distill) against the oracle: generated variables, distillation losses, gradients and
updates of every unit of every stack, and the fused step."""
import numpy as np
import pytest

from conftest import small_cfg
from harness import (GpuRun, NOISE_SEEDS, allowance, log_parity, noisy_bf16_store, oracle_modules, per_tensor_errors, rel_err,
                     to_dev, to_host)
from oracle import lp_oracle as O
from workloads import gen

pytestmark = pytest.mark.gpu


def cfg_f32(K=3):
    if K == 3:
        return small_cfg("preact", N=4, H=8, W=8, stage_channels=(8, 16), stage_blocks=(2, 2), module_block_end=(1, 3, 4))
    return small_cfg("postbn", N=4, H=8, W=8, stage_channels=(8, 16), stage_blocks=(2, 2), module_block_end=(1, 2, 3, 4))


def cfg_bf16():
    return small_cfg("preact", N=16, H=16, W=16, dtype="bf16", stage_channels=(16, 32), stage_blocks=(2, 2),
                     module_block_end=(1, 3, 4), stem_channels=16, classes=10)


@pytest.mark.parametrize("mk,tol", [(lambda: cfg_f32(3), 1e-4), (lambda: cfg_f32(4), 1e-4), (cfg_bf16, 2e-2)])
def test_reauxnet_forward_matches_oracle(mk, tol):
    cfg = mk()
    run = GpuRun(cfg, aux_recursive=True)
    got = run.auxnet()
    net = run.net
    net.store = None if cfg["dtype"] == "f32" else gen.round_bf16
    want = O.reauxnet_forward(net, run.stacks, run.images.astype(np.float64))
    net.store = None
    assert len(got) == net.K - 1
    for k in range(1, net.K):
        assert got[k - 1].shape == tuple(net.boundary[k])
        assert rel_err(got[k - 1], want[k - 1]) < tol, k


def test_shared_parameters_reproduce_the_chain_on_the_gpu():
    """Stacks whose units carry the chain's parameters generate the chain's variables (the paper's
    remark on weight sharing): same kernels, same operands, identical results."""
    cfg = cfg_f32(4)
    chain = GpuRun(cfg)
    want = chain.auxnet()
    rec = GpuRun(cfg, aux_recursive=True)
    for k in range(1, rec.net.K):
        for j in range(k):
            rec.lp.lp_set_params(rec.h, rec.lp.LP_REAUX(k, j), chain.auxs[j])
    got = rec.auxnet()
    for a, b in zip(got, want):
        np.testing.assert_array_equal(a, b)


def test_parameter_layout_and_index_errors():
    cfg = cfg_f32(4)
    run = GpuRun(cfg, aux_recursive=True)
    lp, net = run.lp, run.net
    for k in range(1, net.K):
        for j in range(k):
            lay = lp.lp_param_layout(run.desc, lp.LP_REAUX(k, j))
            assert [(n, tuple(s)) for n, _, s in lay] == [(n, tuple(s)) for n, _, s in net.param_layout(O.LP_AUX(j))]
            np.testing.assert_array_equal(lp.lp_get_params(run.h, lp.LP_REAUX(k, j)), run.stacks[k - 1][j].astype(np.float32))
    with pytest.raises(lp.LpError):
        lp.lp_get_params(run.h, lp.LP_REAUX(net.K, 0))


@pytest.mark.parametrize("mk,tol", [(lambda: cfg_f32(3), 1e-4), (lambda: cfg_f32(4), 1e-4)])
def test_reauxnet_distillation_matches_oracle(mk, tol, lr_lambda=0.05, lr_aux=0.01):
    cfg = mk()
    run = GpuRun(cfg, aux_recursive=True)
    net, lp, torch = run.net, run.lp, run.torch
    K = net.K
    xs_host = run.auxnet()
    run.fwd_bwd_all()
    ref = oracle_modules(run, xs_host)
    d_new = [torch.zeros_like(run.d_x[k]) for k in range(1, K)]
    d_loss = torch.zeros(K - 1, dtype=torch.float32, device="cuda:0")
    lp.lp_auxnet_distill(run.h, run.d_images, run.d_x[1:], run.d_dx, lr_lambda, lr_aux, d_new, d_loss)
    assert lp.lp_last_device_status(run.h) == 0
    newp, newx, losses, grads = O.reauxnet_distill_step(net, run.stacks, run.images.astype(np.float64), xs_host,
                                                       [r["dx"] for r in ref[1:]], [r["seed"] for r in ref[:-1]],
                                                       lr_lambda, lr_aux)
    got_loss = d_loss.cpu().numpy()
    for k in range(1, K):
        assert rel_err(to_host(d_new[k - 1]), newx[k - 1]) < tol, ("x_new", k)
        assert abs(got_loss[k - 1] - losses[k - 1]) < 2 * tol * losses[k - 1], ("loss", k)
        for j in range(k):
            g_gpu = lp.lp_get_grads(run.h, lp.LP_REAUX(k, j))
            errs = per_tensor_errors(net, O.LP_AUX(j), g_gpu, grads[k - 1][j])
            assert max(errs.values()) < 5 * tol, (k, j, errs)
            after = lp.lp_get_params(run.h, lp.LP_REAUX(k, j)).astype(np.float64)
            assert rel_err(after, newp[k - 1][j]) < tol, (k, j)


def test_reauxnet_distillation_bf16_matches_the_storage_model_oracle():
    """bf16: boundaries from the oracle's stacks, dx from the oracle's module passes; losses within 2e-2 (twice
    that for the squared distillation loss), every gradient tensor of every unit within max(2e-2, min(2 x floor,
    0.20)), the floor taken from noisy runs of the oracle's own distillation pass."""
    cfg = cfg_bf16()
    run = GpuRun(cfg, aux_recursive=True)
    net, lp, torch = run.net, run.lp, run.torch
    K = net.K
    images = run.images.astype(np.float64)
    net.store = gen.round_bf16
    ox = O.reauxnet_forward(net, run.stacks, images)
    net.store = None
    gx = run.auxnet()                   # the stacks' kept activations
    for k in range(1, K):
        assert rel_err(gx[k - 1], ox[k - 1]) < 2e-2
    run.set_boundaries(ox)
    xs_host = [to_host(t) for t in run.d_x[1:]]
    run.fwd_bwd_all()
    ref = oracle_modules(run, xs_host)
    d_dx = [None] + [to_dev(ref[k]["dx"], cfg) for k in range(1, K)]
    d_loss = torch.zeros(K - 1, dtype=torch.float32, device="cuda:0")
    lr_lambda, lr_aux = 0.05, 0.01
    lp.lp_auxnet_distill(run.h, run.d_images, run.d_x[1:], d_dx, lr_lambda, lr_aux, None, d_loss)
    assert lp.lp_last_device_status(run.h) == 0
    net.store = gen.round_bf16
    _, newx, losses, grads = O.reauxnet_distill_step(net, run.stacks, images, xs_host, [r["dx"] for r in ref[1:]],
                                                    [r["seed"] for r in ref[:-1]], lr_lambda, lr_aux)
    net.store = None
    floors = {}
    for seed in NOISE_SEEDS:
        net.store = noisy_bf16_store(seed)
        try:
            for k in range(1, K):
                res = O.reauxnet_fwd_bwd(net, k, run.stacks[k - 1], images, newx[k - 1])
                for j in range(k):
                    for n, e in per_tensor_errors(net, O.LP_AUX(j), res["grads"][j], grads[k - 1][j]).items():
                        floors[(k, j, n)] = max(floors.get((k, j, n), 0.0), e)
        finally:
            net.store = None
    got_loss = d_loss.cpu().numpy()
    bad = []
    for k in range(1, K):
        assert abs(got_loss[k - 1] - losses[k - 1]) < 4e-2 * losses[k - 1], (k, got_loss[k - 1], losses[k - 1])
        for j in range(k):
            g = lp.lp_get_grads(run.h, lp.LP_REAUX(k, j)).astype(np.float64)
            for n, e in per_tensor_errors(net, O.LP_AUX(j), g, grads[k - 1][j]).items():
                a = allowance(2e-2, floors[(k, j, n)])
                log_parity(workload=cfg["name"] + " (recursive distillation)", dtype="bf16", module="stack%d/unit%d" % (k, j),
                           tensor=n, err=e, floor=floors[(k, j, n)], allowed=a)
                if not e < a:
                    bad.append((k, j, n, e, floors[(k, j, n)], a))
    assert not bad, bad


def test_fused_step_in_recursive_form_equals_separate_calls():
    cfg = cfg_f32(4)
    a = GpuRun(cfg, aux_recursive=True)
    b = GpuRun(cfg, aux_recursive=True)
    lp, torch = a.lp, a.torch
    K = a.net.K
    lam = a.d_kappa if a.use_kappa else None
    lp.lp_layer_parallel_step(a.h, a.d_images, a.d_x[1:], a.d_labels, lam, cfg["rho"], a.d_loss, a.d_dx, cfg["lr"],
                              0.0, 0.0, cfg["rho"])
    assert lp.lp_last_device_status(a.h) == 0
    b.auxnet()
    b.fwd_bwd_all()
    b.step()
    np.testing.assert_array_equal(a.d_loss.cpu().numpy(), b.d_loss.cpu().numpy())
    for k in range(1, K):
        np.testing.assert_array_equal(to_host(a.d_x[k]), to_host(b.d_x[k]))
        np.testing.assert_array_equal(to_host(a.d_dx[k]), to_host(b.d_dx[k]))
    for k in range(K):   # weight gradients are summed with fp32 atomics: equal up to their order
        np.testing.assert_allclose(lp.lp_get_params(a.h, k), lp.lp_get_params(b.h, k), rtol=1e-5, atol=1e-6)
