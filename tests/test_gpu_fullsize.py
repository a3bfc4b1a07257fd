"""Full-size parity in the launch configuration the benchmark times: the four bf16 workloads at their own
batch sizes, through the grouped call.

The oracle cannot run a whole step at these sizes in seconds, so each workload is checked by properties that
hold at any size -- the penalty vanishes on the feasible set (Section 3.1: psi(x, x) = 0), the augmented-
Lagrangian method with kappa = 0 is the penalty method and its extra terms are linear in kappa (Section 3.2),
the multiplier step c = rho turns kappa into the terminal adjoint, a convolution feeding a batch norm has a
gradient orthogonal to its weights -- and ONE module per workload (the cheapest for the CPU) is compared
with the oracle element by element."""
import numpy as np
import pytest

from harness import GpuRun, allowance, log_parity, noisy_bf16_store, per_tensor_errors, rel_err, to_host, NOISE_SEEDS
from oracle import lp_oracle as O
from workloads import gen, get_config

pytestmark = pytest.mark.gpu

# workload -> module compared with the oracle (the one with the fewest multiply-adds)
ORACLE_MODULE = {"resnet56": 2, "resnet110": 5, "wrn28_10": 3, "resnet34": 3}


@pytest.fixture(scope="module", params=list(ORACLE_MODULE))
def full(request):
    cfg = get_config(request.param)
    cfg["loss"] = "al"                      # exercise the multiplier path; kappa = 0 must equal the penalty
    run = GpuRun(cfg, kappa_std=0.0)
    run.auxnet()                            # boundaries from the GPU AuxNet: only properties are checked on them
    yield run
    run.lp.lp_destroy(run.h)


def test_kappa_zero_equals_penalty_and_loss_is_linear_in_kappa(full):
    run, torch = full, full.torch
    K = run.net.K
    for t in run.d_kappa:
        t.zero_()
    g_al0 = run.fwd_bwd_all()
    loss_al0 = run.d_loss.cpu().numpy().copy()
    run.use_kappa = False
    g_pen = run.fwd_bwd_all()
    loss_pen = run.d_loss.cpu().numpy().copy()
    run.use_kappa = True
    np.testing.assert_allclose(loss_al0, loss_pen, rtol=1e-4)  # fp32 atomics reorder sums between runs
    for k in range(K):
        assert rel_err(g_al0[k], g_pen[k]) < 2e-2      # only the order of fp32 atomic sums differs between the runs
    # L_AL - L_P = <kappa, r>
    r = [torch.zeros_like(run.d_x[k + 1]) for k in range(K - 1)]
    for k in range(K - 1):
        run.lp.lp_get_residual(run.h, k, r[k], None)
        run.d_kappa[k].copy_((0.05 * torch.randn(run.d_kappa[k].shape, device="cuda:0",
                                                 generator=torch.Generator(device="cuda:0").manual_seed(k))).to(torch.bfloat16))
    run.fwd_bwd_all()
    loss_al = run.d_loss.cpu().numpy().copy()
    for k in range(K - 1):
        inner = float((run.d_kappa[k].double() * r[k].double()).sum())
        assert abs((loss_al[k, 0] - loss_pen[k, 0]) - inner) < 2e-2 * abs(inner) + 1e-6 * abs(loss_pen[k, 0])
        np.testing.assert_allclose(loss_al[k, 1], loss_pen[k, 1], rtol=1e-4)
    for t in run.d_kappa:
        t.zero_()


def test_multiplier_step_rho_gives_terminal_adjoint(full):
    run, torch = full, full.torch
    K = run.net.K
    for k in range(K - 1):
        run.d_kappa[k].copy_((0.05 * torch.randn(run.d_kappa[k].shape, device="cuda:0",
                                                 generator=torch.Generator(device="cuda:0").manual_seed(10 + k))).to(torch.bfloat16))
    run.fwd_bwd_all()
    seeds = [torch.zeros_like(run.d_x[k + 1]) for k in range(K - 1)]
    for k in range(K - 1):
        run.lp.lp_get_residual(run.h, k, None, seeds[k])
    params_before = [run.lp.lp_get_params(run.h, k) for k in range(K)]
    run.cfg["lr"] = 0.0
    run.step(kappa_step=run.cfg["rho"])
    for k in range(K - 1):
        assert rel_err(to_host(run.d_kappa[k]), to_host(seeds[k])) < 1e-2
    for k in range(K):                           # lr = 0: the parameters stay where they were
        np.testing.assert_array_equal(run.lp.lp_get_params(run.h, k), params_before[k])
    for t in run.d_kappa:
        t.zero_()


def test_penalty_vanishes_on_the_feasible_set(full):
    """x_{k+1} := F_k(x_k) (rebuilt from the stored residual) leaves a loss and gradients that are rounding
    residue: at least three orders of magnitude below the loss, two below the gradients, of the infeasible point."""
    run, torch = full, full.torch
    K = run.net.K
    run.use_kappa = False
    g0 = run.fwd_bwd_all()
    loss0 = run.d_loss.cpu().numpy().copy()
    saved = [t.clone() for t in run.d_x]
    for k in range(K - 1):
        r = torch.zeros_like(run.d_x[k + 1])
        run.lp.lp_get_residual(run.h, k, r, None)
        # out_k = r + x_{k+1}; the next module's input is not what is tested, only module k's own loss
        feasible = (r.float() + run.d_x[k + 1].float()).to(torch.bfloat16)
        x = list(run.d_x)
        x[k + 1] = feasible
        loss = torch.zeros(2, dtype=torch.float32, device="cuda:0")
        run.lp.lp_module_fwd_bwd(run.h, k, run.d_x[k], feasible, None, run.cfg["rho"], loss, run.d_dx[k])
        assert run.lp.lp_last_device_status(run.h) == 0
        g = run.lp.lp_get_grads(run.h, k)
        assert float(loss[0]) < 1e-3 * loss0[k, 0], (k, float(loss[0]), loss0[k, 0])
        assert np.linalg.norm(g) < 1e-2 * np.linalg.norm(g0[k]), (k, np.linalg.norm(g), np.linalg.norm(g0[k]))
    for a, b in zip(run.d_x, saved):
        a.copy_(b)
    run.use_kappa = True


def test_scale_invariance_of_convs_feeding_a_batch_norm(full):
    """<w, dL/dw> = 0 for a convolution whose output goes straight into a batch norm (eps -> 0)."""
    run = full
    run.fwd_bwd_all()
    desc = run.desc
    checked = 0
    for k in range(run.net.K):
        p = run.lp.lp_get_params(run.h, k).astype(np.float64)
        g = run.lp.lp_get_grads(run.h, k).astype(np.float64)
        off = 0
        for name, kind, shape in run.lp.lp_param_layout(desc, k):
            n = int(np.prod(shape))
            if name.endswith("conv1.w"):
                w, d = p[off:off + n], g[off:off + n]
                assert abs(w @ d) < 2e-2 * np.linalg.norm(w) * np.linalg.norm(d), (k, name)
                checked += 1
            off += n
    assert checked == len(run.net.blocks)


def test_one_module_against_the_oracle_at_full_size(full):
    run = full
    net, cfg = run.net, run.cfg
    k = ORACLE_MODULE[cfg["name"]]
    last = k == net.K - 1
    # inputs of the module from the seeded generator, never from the CUDA path
    xk = gen.round_bf16(gen.normal(7, "x%d" % k, net.boundary[k]))
    run.d_x[k].copy_(run.torch.from_numpy(xk).to("cuda:0").to(run.torch.bfloat16))
    tgt = run.labels
    if not last:
        tgt = gen.round_bf16(gen.normal(7, "x%d" % (k + 1), net.boundary[k + 1]))
        run.d_x[k + 1].copy_(run.torch.from_numpy(tgt).to("cuda:0").to(run.torch.bfloat16))
    for t in run.d_kappa:
        t.zero_()
    run.fwd_bwd_all()
    grads = run.lp.lp_get_grads(run.h, k)
    loss = run.d_loss.cpu().numpy()

    def oracle(store):
        net.store = store
        try:
            return O.module_fwd_bwd(net, k, run.mods[k], xk.astype(np.float64), tgt if last else tgt.astype(np.float64),
                                    None, cfg["rho"])
        finally:
            net.store = None
    ref = oracle(gen.round_bf16)
    fl, fl_dx = {}, 0.0
    for seed in NOISE_SEEDS:
        noisy = oracle(noisy_bf16_store(seed))
        for n, e in per_tensor_errors(net, k, noisy["grads"], ref["grads"]).items():
            fl[n] = max(fl.get(n, 0.0), e)
        fl_dx = max(fl_dx, rel_err(noisy["dx"], ref["dx"]))
    lerr = abs(loss[k, 0] - ref["loss"]) / abs(ref["loss"])
    log_parity(workload=cfg["name"] + " (full size)", dtype="bf16", module=k, tensor="(loss)", err=float(lerr), floor=0.0, allowed=2e-2)
    assert lerr < 2e-2
    errs = per_tensor_errors(net, k, grads, ref["grads"])
    bad = {}
    for n, e in errs.items():
        a = allowance(2e-2, fl[n])
        log_parity(workload=cfg["name"] + " (full size)", dtype="bf16", module=k, tensor=n, err=e, floor=fl[n], allowed=a)
        if not e < a:
            bad[n] = (e, fl[n], a)
    e = rel_err(to_host(run.d_dx[k]), ref["dx"])
    log_parity(workload=cfg["name"] + " (full size)", dtype="bf16", module=k, tensor="(dx)", err=e, floor=fl_dx,
               allowed=allowance(2e-2, fl_dx))
    if not e < allowance(2e-2, fl_dx):
        bad["(dx)"] = (e, fl_dx, allowance(2e-2, fl_dx))
    assert not bad, bad
