"""Helpers shared by the GPU parity tests: run a workload through the C ABI and through the oracle."""
import json
import os

import numpy as np

from oracle import lp_oracle as O
from workloads import gen


def rel_err(a, b):
    a = np.asarray(a, dtype=np.float64).reshape(-1)
    b = np.asarray(b, dtype=np.float64).reshape(-1)
    nb = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / nb) if nb > 0 else float(np.linalg.norm(a))


def torch_dtype(cfg):
    import torch
    return torch.float32 if cfg["dtype"] == "f32" else torch.bfloat16


def to_dev(a, cfg, dev="cuda:0"):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(dev).to(torch_dtype(cfg)).contiguous()


def to_host(t):
    return t.float().cpu().numpy().astype(np.float64)


def make_all_params(net, cfg, perturb=True):
    mods = [gen.make_params(net.param_layout(k), cfg["seed"], "module%d" % k, perturb_bn=perturb, dtype=cfg["dtype"])
            for k in range(net.K)]
    auxs = [gen.make_params(net.param_layout(O.LP_AUX(k)), cfg["seed"], "aux%d" % k, perturb_bn=perturb,
                            dtype=cfg["dtype"]) for k in range(net.K - 1)]
    return mods, auxs


def per_tensor_errors(net, which, got_flat, ref_flat):
    """Relative L2 error of every parameter tensor of a blob.  A tensor whose exact gradient vanishes
    (the shift of a batch norm that only feeds 1x1 convolutions followed by batch norms: the loss does
    not depend on it; the oracle returns rounding noise, below 1e-9 of the blob) has no scale of its
    own: what the GPU returns for it is measured in absolute terms, against the norm of the whole blob.
    fp32 workloads: against 1e-2 of it, so that a tolerance of 1e-4 bounds the tensor at 1e-6 of the
    gradient (cancellation noise of fp32 sums, which varies with the order of the atomic additions).
    bf16 workloads: against the blob norm itself -- with bf16 storage the invariance behind the zero is
    broken at rounding level, and both the GPU and the oracle under rounding noise return about 1e-2 of
    the gradient norm there."""
    out, off = {}, 0
    ref_flat = np.asarray(ref_flat, dtype=np.float64)
    got_flat = np.asarray(got_flat, dtype=np.float64)
    blob = float(np.linalg.norm(ref_flat))
    unit = 1e-2 if net.cfg["dtype"] == "f32" else 1.0
    for name, _, shape in net.param_layout(which):
        n = int(np.prod(shape))
        g, r = got_flat[off:off + n], ref_flat[off:off + n]
        if blob > 0 and np.linalg.norm(r) < 1e-9 * blob:
            out[name] = float(np.linalg.norm(g - r) / (unit * blob))
        else:
            out[name] = rel_err(g, r)
        off += n
    return out


class GpuRun:
    """One workload on the GPU: handle, parameters, device buffers."""

    def __init__(self, cfg, conv_impl=0, perturb=True, kappa_std=None, aux_recursive=False):
        import torch
        import paper_2112_05387_b200 as lp
        self.lp, self.torch, self.cfg = lp, torch, cfg
        self.net = O.Net(cfg)
        self.desc = lp.desc_from_config(cfg, conv_impl, aux_recursive)
        self.h = lp.lp_create(self.desc)
        self.mods, self.auxs = make_all_params(self.net, cfg, perturb)
        for k in range(self.net.K):
            lp.lp_set_params(self.h, k, self.mods[k])
        self.stacks = None
        if aux_recursive:   # stack k = 1..K-1: k units with parameters of their own
            self.stacks = [[gen.make_params(self.net.param_layout(O.LP_AUX(j)), cfg["seed"], "reaux%d/%d" % (k, j),
                                            perturb_bn=perturb, dtype=cfg["dtype"]) for j in range(k)]
                           for k in range(1, self.net.K)]
            for k in range(1, self.net.K):
                for j in range(k):
                    lp.lp_set_params(self.h, lp.LP_REAUX(k, j), self.stacks[k - 1][j])
        else:
            for k in range(self.net.K - 1):
                lp.lp_set_params(self.h, lp.LP_AUX(k), self.auxs[k])
        self.images = gen.make_images(cfg)
        self.labels = gen.make_labels(cfg)
        self.d_images = to_dev(self.images, cfg)
        self.d_labels = torch.from_numpy(self.labels).to("cuda:0")
        K = self.net.K
        self.d_x = [self.d_images] + [torch.zeros(self.net.boundary[k], dtype=torch_dtype(cfg), device="cuda:0")
                                      for k in range(1, K)]
        std = cfg["kappa_std"] if kappa_std is None else kappa_std
        self.kappa = [gen.make_kappa(cfg, k, self.net.boundary[k + 1], std=std) for k in range(K - 1)]
        self.use_kappa = cfg["loss"] == "al"
        self.d_kappa = [to_dev(kp, cfg) for kp in self.kappa]
        self.d_loss = torch.zeros(K, 2, dtype=torch.float32, device="cuda:0")
        self.d_dx = [None] + [torch.zeros_like(self.d_x[k]) for k in range(1, K)]

    def auxnet(self):
        self.lp.lp_auxnet_forward(self.h, self.d_images, self.d_x[1:])
        assert self.lp.lp_last_device_status(self.h) == 0
        return [to_host(t) for t in self.d_x[1:]]

    def set_boundaries(self, xs_host):
        """Load x_1..x_{K-1} from host arrays (oracle AuxNet outputs rounded to the storage type)."""
        for k in range(1, self.net.K):
            self.d_x[k].copy_(to_dev(xs_host[k - 1], self.cfg))

    def fwd_bwd_all(self, grouped=True):
        lp, h = self.lp, self.h
        lam = self.d_kappa if self.use_kappa else None
        if grouped:
            lp.lp_modules_fwd_bwd_all(h, self.d_x, self.d_labels, lam, self.cfg["rho"], self.d_loss, self.d_dx)
        else:
            for k in range(self.net.K):
                last = k == self.net.K - 1
                lp.lp_module_fwd_bwd(h, k, self.d_x[k], self.d_labels if last else self.d_x[k + 1],
                                     None if (last or lam is None) else lam[k], self.cfg["rho"], self.d_loss[k],
                                     self.d_dx[k])
        st = lp.lp_last_device_status(h)
        assert st == 0, lp.lp_status_string(st)
        return [lp.lp_get_grads(h, k) for k in range(self.net.K)]

    def step(self, kappa_step=None):
        lam = self.d_kappa if self.use_kappa else None
        c = self.cfg["rho"] if kappa_step is None else kappa_step
        self.lp.lp_step(self.h, self.cfg["lr"], 0.0, 0.0, c, lam)
        assert self.lp.lp_last_device_status(self.h) == 0


def noisy_bf16_store(seed=1234, eps=1e-7):
    """Storage model with accumulation-order noise: values are perturbed by a relative 1e-7
    (the size of fp32 summation-order effects) before they are rounded to bf16.  Two runs of the
    oracle that differ only by this noise bound how closely ANY bf16-storage implementation can be
    expected to reproduce a gradient tensor: rounding boundaries and ReLU masks turn such noise
    into percent-level changes of the adjoint fields of a deep module."""
    rng = np.random.default_rng(seed)

    def store(a):
        a = np.asarray(a, dtype=np.float64)
        return gen.round_bf16(a * (1.0 + eps * rng.standard_normal(a.shape)))
    return store


# Noise seeds of the floor: the floor of a tensor is the LARGEST change over these runs.
NOISE_SEEDS = (1234, 4321, 777)
# No tensor of a bf16 workload may be further from the oracle than this, whatever its floor.  Measured
# on the CPU alone, the floors of single tensors reach 0.10 - 0.14 in modules of nine basic blocks or
# six bottleneck blocks (the oracle against itself), so a cap below that would reject the oracle too.
ALLOWANCE_CAP = 0.20


def allowance(tol, floor):
    """Largest relative L2 error accepted for a tensor of a bf16 workload: the stated tolerance, widened to
    twice the tensor's own noise floor where that is larger, and never beyond ALLOWANCE_CAP.  (Over all
    recorded comparisons the error of the CUDA path is 0.97 x the floor in the median and 1.41 x at most.)"""
    return max(tol, min(2.0 * floor, ALLOWANCE_CAP))


def log_parity(**rec):
    """Append one record (tensor, error, floor, allowance) to the file named by LP_PARITY_LOG, if set."""
    path = os.environ.get("LP_PARITY_LOG")
    if not path:
        return
    rec["test"] = os.environ.get("PYTEST_CURRENT_TEST", "").split(" ")[0]
    with open(path, "a") as f:
        f.write(json.dumps(rec) + "\n")


def noise_floors(run, xs_host, ref, kappas=None, params=None):
    """Per module: the noise floor of every gradient tensor, of the whole gradient and of dx -- the largest
    relative change between the storage-model oracle `ref` and runs of the same oracle that differ only by
    rounding-level noise before each bf16 rounding (one run per seed in NOISE_SEEDS)."""
    net = run.net
    floors = [dict(grads={}, whole=0.0, dx=0.0) for _ in range(net.K)]
    for seed in NOISE_SEEDS:
        noisy = oracle_modules(run, xs_host, kappas=kappas, params=params, store=noisy_bf16_store(seed))
        for k in range(net.K):
            per = per_tensor_errors(net, k, noisy[k]["grads"], ref[k]["grads"])
            for n, e in per.items():
                floors[k]["grads"][n] = max(floors[k]["grads"].get(n, 0.0), e)
            floors[k]["whole"] = max(floors[k]["whole"], rel_err(noisy[k]["grads"], ref[k]["grads"]))
            if ref[k]["dx"] is not None:
                floors[k]["dx"] = max(floors[k]["dx"], rel_err(noisy[k]["dx"], ref[k]["dx"]))
    return floors


def oracle_modules(run, xs_host, kappas=None, params=None, exact=False, store=None):
    """Oracle module_fwd_bwd for every module on the given boundary tensors (x_0 = images).

    For a bf16 workload the oracle rounds activations where the step stores them (unless
    ``exact``): ReLU masks and max-pool winners are decisions taken by floating point, and both
    sides must take them on the same values -- exact arithmetic alone moves gradient tensors of a
    randomly initialised network by several percent through flipped masks."""
    net, cfg = run.net, run.cfg
    net.store = None if (exact or cfg["dtype"] == "f32") else (store or gen.round_bf16)
    xs = [run.images.astype(np.float64)] + [np.asarray(x, dtype=np.float64) for x in xs_host]
    params = run.mods if params is None else params
    kappas = (run.kappa if run.use_kappa else None) if kappas is None else kappas
    out = []
    for k in range(net.K):
        last = k == net.K - 1
        out.append(O.module_fwd_bwd(net, k, params[k], xs[k], run.labels if last else xs[k + 1],
                                    None if (last or kappas is None) else kappas[k], cfg["rho"]))
    net.store = None
    return out
