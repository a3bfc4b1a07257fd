"""CPU oracle for the layer-parallel training step (TEST INFRASTRUCTURE ONLY).

A plain, slow, fp64 numpy statement of what one step of the paper's
layer-parallel method computes: AuxNet forward chain (Eq. AV-Net-FP-lambda,
Algorithm 1 first loop), decoupled module forward (Eq.
Parallel-ResNet-Feature-Flow), penalty / augmented-Lagrangian local loss with
its terminal adjoint (Eq. Parallel-ResNet-Gradient-Propagation-Equation, AL
functional of Section 3), module back-propagation (Eq.
Parallel-ResNet-Backpropagation), and the SGD / multiplier update (Eq.
Parallel-ResNet-Multiplier-Update).  Every operator is its textbook definition;
a matrix product per filter tap is the only library primitive used.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It shares no code with the CUDA path and imports nothing from it.
All parts are pinned by tests/test_oracle_*.py (brute force, adjoint
identities, finite differences, closed forms, the paper's own invariants).

Layout: activations NHWC, convolution weights [C_out, R, S, C_in], linear
weights [classes, C].  Penalty coefficient: the paper's beta*||.||^2 is written
(rho/2)*||.||^2, rho = 2*beta.  The multiplier attached to the constraint
F_k(x_k) = x_{k+1} is the paper's kappa_{k+1}.
"""
import numpy as np

F = np.float64


# ----------------------------------------------------------------------------
# operators (definitions)
# ----------------------------------------------------------------------------
def out_size(h, r, stride, pad):
    return (h + 2 * pad - r) // stride + 1


def conv_fwd(x, w, stride, pad):
    """Cross-correlation y[n,oh,ow,co] = sum_{r,s,ci} w[co,r,s,ci] x[n,oh*st+r-p,ow*st+s-p,ci]."""
    n, h, wd, ci = x.shape
    co, R, S, ci2 = w.shape
    assert ci == ci2
    oh, ow = out_size(h, R, stride, pad), out_size(wd, S, stride, pad)
    xp = np.zeros((n, h + 2 * pad, wd + 2 * pad, ci), dtype=F)
    xp[:, pad:pad + h, pad:pad + wd, :] = x
    y = np.zeros((n * oh * ow, co), dtype=F)
    for r in range(R):
        for s in range(S):
            xs = xp[:, r:r + stride * (oh - 1) + 1:stride, s:s + stride * (ow - 1) + 1:stride, :]
            y += xs.reshape(-1, ci) @ w[:, r, s, :].T
    return y.reshape(n, oh, ow, co)


def conv_dgrad(dy, w, stride, pad, x_shape):
    """Gradient of <conv_fwd(x,w), dy> with respect to x."""
    n, h, wd, ci = x_shape
    co, R, S, _ = w.shape
    _, oh, ow, _ = dy.shape
    dxp = np.zeros((n, h + 2 * pad, wd + 2 * pad, ci), dtype=F)
    d2 = dy.reshape(-1, co)
    for r in range(R):
        for s in range(S):
            contrib = (d2 @ w[:, r, s, :]).reshape(n, oh, ow, ci)
            dxp[:, r:r + stride * (oh - 1) + 1:stride, s:s + stride * (ow - 1) + 1:stride, :] += contrib
    return dxp[:, pad:pad + h, pad:pad + wd, :].copy()


def conv_wgrad(x, dy, w_shape, stride, pad):
    """Gradient of <conv_fwd(x,w), dy> with respect to w."""
    n, h, wd, ci = x.shape
    co, R, S, _ = w_shape
    _, oh, ow, _ = dy.shape
    xp = np.zeros((n, h + 2 * pad, wd + 2 * pad, ci), dtype=F)
    xp[:, pad:pad + h, pad:pad + wd, :] = x
    d2 = dy.reshape(-1, co)
    dw = np.zeros(w_shape, dtype=F)
    for r in range(R):
        for s in range(S):
            xs = xp[:, r:r + stride * (oh - 1) + 1:stride, s:s + stride * (ow - 1) + 1:stride, :]
            dw[:, r, s, :] = d2.T @ xs.reshape(-1, ci)
    return dw


def bn_fwd(x, gamma, beta, eps):
    """Training-mode batch normalisation over (N,H,W) per channel, biased variance."""
    mean = x.mean(axis=(0, 1, 2))
    var = ((x - mean) ** 2).mean(axis=(0, 1, 2))
    rstd = 1.0 / np.sqrt(var + eps)
    xhat = (x - mean) * rstd
    return gamma * xhat + beta, (xhat, rstd)


def bn_bwd(dy, cache, gamma):
    xhat, rstd = cache
    m = dy.shape[0] * dy.shape[1] * dy.shape[2]
    dbeta = dy.sum(axis=(0, 1, 2))
    dgamma = (dy * xhat).sum(axis=(0, 1, 2))
    dx = (gamma * rstd) * (dy - dbeta / m - xhat * (dgamma / m))
    return dx, dgamma, dbeta


def relu(x):
    return np.where(x > 0, x, 0.0)


def relu_bwd(dy, x):
    """ReLU'(0) = 0."""
    return np.where(x > 0, dy, 0.0)


def maxpool_fwd(x, k=3, stride=2, pad=1):
    """Max over k x k windows; padding cells are -inf; first maximum in (h,w) scan order wins."""
    n, h, w, c = x.shape
    oh, ow = out_size(h, k, stride, pad), out_size(w, k, stride, pad)
    xp = np.full((n, h + 2 * pad, w + 2 * pad, c), -np.inf, dtype=F)
    xp[:, pad:pad + h, pad:pad + w, :] = x
    best = np.full((n, oh, ow, c), -np.inf, dtype=F)
    arg = np.zeros((n, oh, ow, c), dtype=np.int64)
    for r in range(k):
        for s in range(k):
            v = xp[:, r:r + stride * (oh - 1) + 1:stride, s:s + stride * (ow - 1) + 1:stride, :]
            better = v > best                      # strict: the first maximum is kept
            best = np.where(better, v, best)
            arg = np.where(better, r * k + s, arg)
    return best, (arg, x.shape, k, stride, pad)


def maxpool_bwd(dy, cache):
    arg, x_shape, k, stride, pad = cache
    n, h, w, c = x_shape
    _, oh, ow, _ = dy.shape
    dxp = np.zeros((n, h + 2 * pad, w + 2 * pad, c), dtype=F)
    for r in range(k):
        for s in range(k):
            sel = np.where(arg == r * k + s, dy, 0.0)
            dxp[:, r:r + stride * (oh - 1) + 1:stride, s:s + stride * (ow - 1) + 1:stride, :] += sel
    return dxp[:, pad:pad + h, pad:pad + w, :].copy()


def avgpool_fwd(x):
    return x.mean(axis=(1, 2))


def avgpool_bwd(dy, x_shape):
    n, h, w, c = x_shape
    return np.broadcast_to(dy[:, None, None, :] / (h * w), x_shape).astype(F)


def linear_fwd(x, w, b):
    return x @ w.T + b


def softmax_ce(logits, labels):
    """Mean over the batch of -log softmax(logits)[label]; gradient (softmax - onehot)/N."""
    n = logits.shape[0]
    z = logits - logits.max(axis=1, keepdims=True)
    lse = np.log(np.exp(z).sum(axis=1, keepdims=True))
    logp = z - lse
    loss = -logp[np.arange(n), labels].mean()
    g = np.exp(logp)
    g[np.arange(n), labels] -= 1.0
    return loss, g / n


def local_loss(out, x_next, kappa, rho):
    """Interior local loss (rho/2)||r||^2 + <kappa, r>, r = out - x_next, and its terminal adjoint."""
    r = out - x_next
    rn2 = float((r * r).sum())
    loss = 0.5 * rho * rn2
    seed = rho * r
    if kappa is not None:
        loss += float((kappa * r).sum())
        seed = seed + kappa
    return loss, rn2, r, seed


# ----------------------------------------------------------------------------
# network structure (derived from a workload dict)
# ----------------------------------------------------------------------------
AUX_BASE = 256


def LP_AUX(k):
    return AUX_BASE + k


class Net:
    """Static structure of one workload: blocks, module split, boundaries, parameter layouts."""

    def __init__(self, cfg):
        self.cfg = cfg
        # Optional model of activation storage: a callable applied wherever the step keeps an
        # activation or adjoint tensor between operators.  None (default) = exact arithmetic.
        # Tests of reduced-precision storage pass a rounding function so that the decisions that
        # floating point takes (ReLU masks, max-pool winners) are taken on the same values.
        self.store = None
        self.K = len(cfg["module_block_end"])
        self.eps = float(cfg["bn_eps"])
        self.kind = cfg["block_kind"]
        assert self.kind in ("postbn", "preact", "bottleneck")
        # the bottleneck block is a post-activation block with three convolutions: stem, head and the
        # storage of block outputs follow the post-BN form
        self.post = self.kind in ("postbn", "bottleneck")
        # stem output geometry
        h, w = cfg["H"], cfg["W"]
        if cfg["stem_kind"] == "conv3x3":
            self.stem = dict(R=3, stride=1, pad=1, pool=False)
        else:
            self.stem = dict(R=7, stride=2, pad=3, pool=True)
            h, w = out_size(h, 7, 2, 3), out_size(w, 7, 2, 3)
            h, w = out_size(h, 3, 2, 1), out_size(w, 3, 2, 1)
        c = cfg["stem_channels"]
        self.blocks = []
        for ch, nb, st in zip(cfg["stage_channels"], cfg["stage_blocks"], cfg["stage_stride"]):
            for b in range(nb):
                s = st if b == 0 else 1
                blk = dict(cin=c, cout=ch, stride=s, hin=h, win=w, proj=(s != 1 or c != ch), mid=ch // 4)
                h, w = out_size(h, 3, s, 1), out_size(w, 3, s, 1)
                blk["hout"], blk["wout"] = h, w
                self.blocks.append(blk)
                c = ch
        ends = list(cfg["module_block_end"])
        assert ends[-1] == len(self.blocks)
        self.module_blocks = [list(range(a, b)) for a, b in zip([0] + ends[:-1], ends)]
        # boundary shapes: x_0 is the image batch, x_k the input of module k
        self.boundary = [(cfg["N"], cfg["H"], cfg["W"], cfg["C_in"])]
        for k in range(1, self.K):
            b = self.blocks[self.module_blocks[k][0]]
            self.boundary.append((cfg["N"], b["hin"], b["win"], b["cin"]))
        # AuxNet_k : x_k -> x_{k+1}
        self.aux = []
        for k in range(self.K - 1):
            _, hi, wi, ci = self.boundary[k]
            _, ho, wo, co = self.boundary[k + 1]
            total = hi // ho
            assert total in (1, 2, 4) and hi == ho * total
            if cfg["aux_convs"] == 1:
                assert total in (1, 2)
                convs = [dict(cin=ci, cout=co, stride=total)]
            else:
                hid = max(co // cfg["aux_width_div"], 1)
                s1 = 2 if total >= 2 else 1
                s2 = 2 if total == 4 else 1
                convs = [dict(cin=ci, cout=hid, stride=s1), dict(cin=hid, cout=co, stride=s2)]
            self.aux.append(convs)

    # -- parameter layouts: list of (name, kind, shape) in blob order -----------
    def param_layout(self, which):
        L = []
        if which >= AUX_BASE:
            for i, cv in enumerate(self.aux[which - AUX_BASE]):
                L.append(("conv%d.w" % (i + 1), "conv_w", (cv["cout"], 3, 3, cv["cin"])))
                L.append(("bn%d.g" % (i + 1), "bn_gamma", (cv["cout"],)))
                L.append(("bn%d.b" % (i + 1), "bn_beta", (cv["cout"],)))
            return L
        k = which
        cfg = self.cfg
        if k == 0:
            R = self.stem["R"]
            L.append(("stem.conv.w", "conv_w", (cfg["stem_channels"], R, R, cfg["C_in"])))
            if self.post:
                L.append(("stem.bn.g", "bn_gamma", (cfg["stem_channels"],)))
                L.append(("stem.bn.b", "bn_beta", (cfg["stem_channels"],)))
        for bi in self.module_blocks[k]:
            b = self.blocks[bi]
            p = "block%d." % bi
            ci, co = b["cin"], b["cout"]
            if self.kind == "bottleneck":
                m = b["mid"]
                L += [(p + "conv1.w", "conv_w", (m, 1, 1, ci)), (p + "bn1.g", "bn_gamma", (m,)), (p + "bn1.b", "bn_beta", (m,)),
                      (p + "conv2.w", "conv_w", (m, 3, 3, m)), (p + "bn2.g", "bn_gamma", (m,)), (p + "bn2.b", "bn_beta", (m,)),
                      (p + "conv3.w", "conv_w", (co, 1, 1, m)), (p + "bn3.g", "bn_gamma", (co,)), (p + "bn3.b", "bn_beta", (co,))]
                if b["proj"]:
                    L += [(p + "sc.w", "conv_w", (co, 1, 1, ci)), (p + "bns.g", "bn_gamma", (co,)),
                          (p + "bns.b", "bn_beta", (co,))]
            elif self.kind == "postbn":
                L += [(p + "conv1.w", "conv_w", (co, 3, 3, ci)), (p + "bn1.g", "bn_gamma", (co,)),
                      (p + "bn1.b", "bn_beta", (co,)),
                      (p + "conv2.w", "conv_w", (co, 3, 3, co)), (p + "bn2.g", "bn_gamma", (co,)),
                      (p + "bn2.b", "bn_beta", (co,))]
                if b["proj"]:
                    L += [(p + "sc.w", "conv_w", (co, 1, 1, ci)), (p + "bns.g", "bn_gamma", (co,)),
                          (p + "bns.b", "bn_beta", (co,))]
            else:
                L += [(p + "bn1.g", "bn_gamma", (ci,)), (p + "bn1.b", "bn_beta", (ci,)),
                      (p + "conv1.w", "conv_w", (co, 3, 3, ci)),
                      (p + "bn2.g", "bn_gamma", (co,)), (p + "bn2.b", "bn_beta", (co,)),
                      (p + "conv2.w", "conv_w", (co, 3, 3, co))]
                if b["proj"]:
                    L.append((p + "sc.w", "conv_w", (co, 1, 1, ci)))
        if k == self.K - 1:
            c = self.blocks[-1]["cout"]
            if self.kind == "preact":
                L += [("head.bn.g", "bn_gamma", (c,)), ("head.bn.b", "bn_beta", (c,))]
            L += [("head.fc.w", "fc_w", (cfg["num_classes"], c)), ("head.fc.b", "fc_b", (cfg["num_classes"],))]
        return L

    def param_count(self, which):
        return int(sum(np.prod(s) for _, _, s in self.param_layout(which)))

    def unpack(self, which, flat):
        flat = np.asarray(flat, dtype=F)
        out, off = {}, 0
        for name, _, shape in self.param_layout(which):
            n = int(np.prod(shape))
            out[name] = flat[off:off + n].reshape(shape)
            off += n
        assert off == flat.size, (off, flat.size)
        return out

    def pack(self, which, named):
        return np.concatenate([np.asarray(named[name], dtype=F).reshape(-1)
                               for name, _, _ in self.param_layout(which)])


def _st(net, a):
    return a if net.store is None else np.asarray(net.store(a), dtype=F)


def _wq(net, w):
    """Convolution weights as the contraction reads them (the storage model also applies to the
    operand copy of the weights; the fp32 master that the update touches is not rounded)."""
    return _st(net, w)


# ----------------------------------------------------------------------------
# AuxNet forward chain  (Eq. AV-Net-FP-lambda; Algorithm 1, first inner loop)
# ----------------------------------------------------------------------------
def auxnet_apply(net, k, p, x):
    """x_{k+1} = AuxNet_k(x_k): conv3x3-BN[-ReLU-conv3x3-BN], batch statistics, no final ReLU."""
    convs = net.aux[k]
    h = _st(net, conv_fwd(x, _wq(net, p["conv1.w"]), convs[0]["stride"], 1))
    h, _ = bn_fwd(h, p["bn1.g"], p["bn1.b"], net.eps)
    if len(convs) == 2:
        h = _st(net, relu(h))
        h = _st(net, conv_fwd(h, _wq(net, p["conv2.w"]), convs[1]["stride"], 1))
        h, _ = bn_fwd(h, p["bn2.g"], p["bn2.b"], net.eps)
    return _st(net, h)


def auxnet_fwd_bwd(net, k, params_flat, x_in, target):
    """Distillation loss D = ||target - AuxNet_k(x_in)||^2 (Eq. AV-Net-lambda: `target` is the
    corrected auxiliary variable, held constant) and its gradient with respect to AuxNet_k's
    parameters.  Returns dict(out, loss, grads (flat, blob order))."""
    p = net.unpack(LP_AUX(k), params_flat)
    convs = net.aux[k]
    x_in = np.asarray(x_in, dtype=F)
    y1 = _st(net, conv_fwd(x_in, _wq(net, p["conv1.w"]), convs[0]["stride"], 1))
    z1, c1 = bn_fwd(y1, p["bn1.g"], p["bn1.b"], net.eps)
    g = {}
    if len(convs) == 2:
        h = _st(net, relu(z1))
        y2 = _st(net, conv_fwd(h, _wq(net, p["conv2.w"]), convs[1]["stride"], 1))
        z2, c2 = bn_fwd(y2, p["bn2.g"], p["bn2.b"], net.eps)
        out = _st(net, z2)
    else:
        out = _st(net, z1)
    diff = out - np.asarray(target, dtype=F)
    loss = float((diff * diff).sum())
    d = _st(net, 2.0 * diff)
    if len(convs) == 2:
        dy2, g["bn2.g"], g["bn2.b"] = bn_bwd(d, c2, p["bn2.g"])
        dy2 = _st(net, dy2)
        g["conv2.w"] = conv_wgrad(h, dy2, p["conv2.w"].shape, convs[1]["stride"], 1)
        dh = _st(net, conv_dgrad(dy2, _wq(net, p["conv2.w"]), convs[1]["stride"], 1, h.shape))
        d = relu_bwd(dh, z1)
    dy1, g["bn1.g"], g["bn1.b"] = bn_bwd(d, c1, p["bn1.g"])
    dy1 = _st(net, dy1)
    g["conv1.w"] = conv_wgrad(x_in, dy1, p["conv1.w"].shape, convs[0]["stride"], 1)
    return dict(out=out, loss=loss, grads=net.pack(LP_AUX(k), g))


def aux_correction(x_k, dx_k, seed_prev, lr_lambda):
    """Correction of the auxiliary variable x_k (Eq. Parallel-ResNet-Slack-Variables-Update):
    x_k <- x_k - lr * (P^k_{kn} + beta dpsi(x_k, out_{k-1})/dx_k - kappa_k).  With psi the squared
    l2 norm and beta = rho/2 the last two terms are -(rho r_{k-1} + kappa_k), minus the terminal
    adjoint of module k-1, so the direction is g_k = dx_k - seed_{k-1}."""
    g = np.asarray(dx_k, dtype=F) - np.asarray(seed_prev, dtype=F)
    return np.asarray(x_k, dtype=F) - lr_lambda * g, g


def auxnet_distill_step(net, aux_params, images, xs, dxs, seeds, lr_lambda, lr_aux):
    """Second parallel loop of Algorithm 1 for every boundary k = 1..K-1: correct x_k, then one SGD
    step of AuxNet_{k-1} on ||x_k_new - AuxNet_{k-1}(x_{k-1})||^2 (x_{k-1} and x_k_new constant).
    xs[k-1] = x_k, dxs[k-1] = dx_k, seeds[k-1] = terminal adjoint of module k-1."""
    new_params, new_x, losses, grads = [], [], [], []
    for k in range(1, net.K):
        x_new, _ = aux_correction(xs[k - 1], dxs[k - 1], seeds[k - 1], lr_lambda)
        x_in = images if k == 1 else xs[k - 2]
        res = auxnet_fwd_bwd(net, k - 1, aux_params[k - 1], x_in, x_new)
        new_params.append(sgd_update(aux_params[k - 1], res["grads"], lr_aux)[0])
        new_x.append(x_new)
        losses.append(res["loss"])
        grads.append(res["grads"])
    return new_params, new_x, losses, grads


def auxnet_forward(net, aux_params, images, post=None):
    """Serial chain x_0 = images, x_{k+1} = AuxNet_k(x_k).  ``post`` (optional) is applied to
    each x_{k+1} before it feeds the next AuxNet (tests use it to model storage rounding)."""
    xs, x = [], np.asarray(images, dtype=F)
    for k in range(net.K - 1):
        x = auxnet_apply(net, k, net.unpack(LP_AUX(k), aux_params[k]), x)
        if post is not None:
            x = np.asarray(post(x), dtype=F)
        xs.append(x)
    return xs


# ----------------------------------------------------------------------------
# Recursive auxiliary-variable networks  (Section 4.3, "Recursive Auxiliary-Variable Networks":
# Eq. ReAuxNet-FP and Eq. ReAuxNet-Distill)
#
# ReAuxNet_k(X_0; xi_k) = AuxNet_{k-1}(AuxNet_{k-2}(... AuxNet_0(X_0) ...)) with parameters xi_k of
# its own: a stack of k units, unit j having the architecture of AuxNet_j.  Every x_k, k = 1..K-1,
# is generated from the input batch alone, so the K-1 stacks are independent of one another.
# ``stacks[k-1]`` is the list of the k flat parameter blobs of stack k (unit j in AuxNet_j's layout).
# ----------------------------------------------------------------------------
def _aux_unit_fwd(net, j, p, x):
    """One AuxNet-shaped unit, keeping what its backward pass needs."""
    convs = net.aux[j]
    c = {"x": x}
    c["y1"] = _st(net, conv_fwd(x, _wq(net, p["conv1.w"]), convs[0]["stride"], 1))
    c["z1"], c["bn1"] = bn_fwd(c["y1"], p["bn1.g"], p["bn1.b"], net.eps)
    if len(convs) == 2:
        c["h"] = _st(net, relu(c["z1"]))
        c["y2"] = _st(net, conv_fwd(c["h"], _wq(net, p["conv2.w"]), convs[1]["stride"], 1))
        c["z2"], c["bn2"] = bn_fwd(c["y2"], p["bn2.g"], p["bn2.b"], net.eps)
        return _st(net, c["z2"]), c
    return _st(net, c["z1"]), c


def _aux_unit_bwd(net, j, p, c, d, need_dx):
    """Adjoint d of the unit's output -> parameter gradients (dict) and, on request, the adjoint of
    its input."""
    convs = net.aux[j]
    g = {}
    if len(convs) == 2:
        dy2, g["bn2.g"], g["bn2.b"] = bn_bwd(d, c["bn2"], p["bn2.g"])
        dy2 = _st(net, dy2)
        g["conv2.w"] = conv_wgrad(c["h"], dy2, p["conv2.w"].shape, convs[1]["stride"], 1)
        dh = _st(net, conv_dgrad(dy2, _wq(net, p["conv2.w"]), convs[1]["stride"], 1, c["h"].shape))
        d = relu_bwd(dh, c["z1"])
    dy1, g["bn1.g"], g["bn1.b"] = bn_bwd(d, c["bn1"], p["bn1.g"])
    dy1 = _st(net, dy1)
    g["conv1.w"] = conv_wgrad(c["x"], dy1, p["conv1.w"].shape, convs[0]["stride"], 1)
    dx = _st(net, conv_dgrad(dy1, _wq(net, p["conv1.w"]), convs[0]["stride"], 1, c["x"].shape)) if need_dx else None
    return g, dx


def reauxnet_forward(net, stacks, images):
    """x_k = ReAuxNet_k(X_0; xi_k) for k = 1..K-1 (Eq. ReAuxNet-FP), each from the images alone."""
    xs = []
    for k in range(1, net.K):
        x = np.asarray(images, dtype=F)
        for j in range(k):
            x, _ = _aux_unit_fwd(net, j, net.unpack(LP_AUX(j), stacks[k - 1][j]), x)
        xs.append(x)
    return xs


def reauxnet_fwd_bwd(net, k, stack_params, images, target):
    """D = ||target - ReAuxNet_k(X_0)||^2 and its gradient with respect to every unit of stack k
    (``target`` constant).  Returns dict(out, loss, grads: list of k flat blobs)."""
    ps = [net.unpack(LP_AUX(j), stack_params[j]) for j in range(k)]
    x, caches = np.asarray(images, dtype=F), []
    for j in range(k):
        x, c = _aux_unit_fwd(net, j, ps[j], x)
        caches.append(c)
    diff = x - np.asarray(target, dtype=F)
    loss = float((diff * diff).sum())
    d = _st(net, 2.0 * diff)
    grads = [None] * k
    for j in range(k - 1, -1, -1):
        g, d = _aux_unit_bwd(net, j, ps[j], caches[j], d, need_dx=j > 0)
        grads[j] = net.pack(LP_AUX(j), g)
    return dict(out=x, loss=loss, grads=grads)


def reauxnet_distill_step(net, stacks, images, xs, dxs, seeds, lr_lambda, lr_aux):
    """Knowledge distillation of the recursive networks (Eq. ReAuxNet-Distill), in the same form as
    ``auxnet_distill_step``: the direction g_k = dx_k - seed_{k-1} (adjoint at the module input plus
    the derivative of the penalty with respect to x_k) corrects x_k, and every unit of stack k takes
    one SGD step on ||x_k_new - ReAuxNet_k(X_0)||^2.  With x_k just generated by the stack this
    gradient is 2*lr_lambda * g_k dReAuxNet_k/dxi_k, the direction of the paper's update."""
    new_stacks, new_x, losses, grads = [], [], [], []
    for k in range(1, net.K):
        x_new, _ = aux_correction(xs[k - 1], dxs[k - 1], seeds[k - 1], lr_lambda)
        res = reauxnet_fwd_bwd(net, k, stacks[k - 1], images, x_new)
        new_stacks.append([sgd_update(stacks[k - 1][j], res["grads"][j], lr_aux)[0] for j in range(k)])
        new_x.append(x_new)
        losses.append(res["loss"])
        grads.append(res["grads"])
    return new_stacks, new_x, losses, grads


# ----------------------------------------------------------------------------
# module forward / backward
# ----------------------------------------------------------------------------
def _stem_fwd(net, p, x, cache):
    st = net.stem
    y = _st(net, conv_fwd(x, _wq(net, p["stem.conv.w"]), st["stride"], st["pad"]))
    cache["stem.x"] = x
    if net.post:
        z, cache["stem.bn"] = bn_fwd(y, p["stem.bn.g"], p["stem.bn.b"], net.eps)
        cache["stem.z"] = z
        y = _st(net, relu(z))
        if st["pool"]:
            y, cache["stem.pool"] = maxpool_fwd(y)
    return y


def _stem_bwd(net, p, d, cache, g):
    st = net.stem
    if net.post:
        if st["pool"]:
            d = _st(net, maxpool_bwd(d, cache["stem.pool"]))
        d = relu_bwd(d, cache["stem.z"])
        d, g["stem.bn.g"], g["stem.bn.b"] = bn_bwd(d, cache["stem.bn"], p["stem.bn.g"])
        d = _st(net, d)
    g["stem.conv.w"] = conv_wgrad(cache["stem.x"], d, p["stem.conv.w"].shape, st["stride"], st["pad"])
    return None        # the gradient with respect to the image is not used


def _block_fwd(net, bi, p, x, cache):
    """One residual block X + F(X, W) (Eq. ResNet-Training-Task), either block form."""
    b = net.blocks[bi]
    q = "block%d." % bi
    c = cache.setdefault(bi, {})
    c["x"] = x
    if net.kind == "bottleneck":
        # conv1x1 - BN - ReLU - conv3x3 (carries the stride) - BN - ReLU - conv1x1 - BN, plus shortcut
        y1 = _st(net, conv_fwd(x, _wq(net, p[q + "conv1.w"]), 1, 0))
        z1, c["bn1"] = bn_fwd(y1, p[q + "bn1.g"], p[q + "bn1.b"], net.eps)
        a1 = _st(net, relu(z1))
        y2 = _st(net, conv_fwd(a1, _wq(net, p[q + "conv2.w"]), b["stride"], 1))
        z2, c["bn2"] = bn_fwd(y2, p[q + "bn2.g"], p[q + "bn2.b"], net.eps)
        a2 = _st(net, relu(z2))
        y3 = _st(net, conv_fwd(a2, _wq(net, p[q + "conv3.w"]), 1, 0))
        z3, c["bn3"] = bn_fwd(y3, p[q + "bn3.g"], p[q + "bn3.b"], net.eps)
        c["z1"], c["a1"], c["z2"], c["a2"] = z1, a1, z2, a2
        if b["proj"]:
            ys = _st(net, conv_fwd(x, _wq(net, p[q + "sc.w"]), b["stride"], 0))
            sc, c["bns"] = bn_fwd(ys, p[q + "bns.g"], p[q + "bns.b"], net.eps)
        else:
            sc = x
        return sc + z3
    if net.kind == "postbn":
        y1 = _st(net, conv_fwd(x, _wq(net, p[q + "conv1.w"]), b["stride"], 1))
        z1, c["bn1"] = bn_fwd(y1, p[q + "bn1.g"], p[q + "bn1.b"], net.eps)
        a1 = _st(net, relu(z1))
        y2 = _st(net, conv_fwd(a1, _wq(net, p[q + "conv2.w"]), 1, 1))
        z2, c["bn2"] = bn_fwd(y2, p[q + "bn2.g"], p[q + "bn2.b"], net.eps)
        c["z1"], c["a1"] = z1, a1
        if b["proj"]:
            ys = _st(net, conv_fwd(x, _wq(net, p[q + "sc.w"]), b["stride"], 0))
            sc, c["bns"] = bn_fwd(ys, p[q + "bns.g"], p[q + "bns.b"], net.eps)
        else:
            sc = x
        return sc + z2
    # pre-activation form
    z0, c["bn1"] = bn_fwd(x, p[q + "bn1.g"], p[q + "bn1.b"], net.eps)
    o = _st(net, relu(z0))
    y1 = _st(net, conv_fwd(o, _wq(net, p[q + "conv1.w"]), b["stride"], 1))
    z1, c["bn2"] = bn_fwd(y1, p[q + "bn2.g"], p[q + "bn2.b"], net.eps)
    a1 = _st(net, relu(z1))
    y2 = conv_fwd(a1, _wq(net, p[q + "conv2.w"]), 1, 1)
    c["z0"], c["o"], c["z1"], c["a1"] = z0, o, z1, a1
    sc = _st(net, conv_fwd(o, _wq(net, p[q + "sc.w"]), b["stride"], 0)) if b["proj"] else x
    return sc + y2


def _block_bwd(net, bi, p, d, cache, g):
    """Adjoint step P_m = P_{m+1} dX_{m+1}/dX_m and the block's parameter gradients."""
    b = net.blocks[bi]
    q = "block%d." % bi
    c = cache[bi]
    x = c["x"]
    if net.kind == "bottleneck":
        dy3, g[q + "bn3.g"], g[q + "bn3.b"] = bn_bwd(d, c["bn3"], p[q + "bn3.g"])
        dy3 = _st(net, dy3)
        g[q + "conv3.w"] = conv_wgrad(c["a2"], dy3, p[q + "conv3.w"].shape, 1, 0)
        da2 = _st(net, conv_dgrad(dy3, _wq(net, p[q + "conv3.w"]), 1, 0, c["a2"].shape))
        dz2 = relu_bwd(da2, c["z2"])
        dy2, g[q + "bn2.g"], g[q + "bn2.b"] = bn_bwd(dz2, c["bn2"], p[q + "bn2.g"])
        dy2 = _st(net, dy2)
        g[q + "conv2.w"] = conv_wgrad(c["a1"], dy2, p[q + "conv2.w"].shape, b["stride"], 1)
        da1 = _st(net, conv_dgrad(dy2, _wq(net, p[q + "conv2.w"]), b["stride"], 1, c["a1"].shape))
        dz1 = relu_bwd(da1, c["z1"])
        dy1, g[q + "bn1.g"], g[q + "bn1.b"] = bn_bwd(dz1, c["bn1"], p[q + "bn1.g"])
        dy1 = _st(net, dy1)
        g[q + "conv1.w"] = conv_wgrad(x, dy1, p[q + "conv1.w"].shape, 1, 0)
        dx = conv_dgrad(dy1, _wq(net, p[q + "conv1.w"]), 1, 0, x.shape)
        if b["proj"]:
            dys, g[q + "bns.g"], g[q + "bns.b"] = bn_bwd(d, c["bns"], p[q + "bns.g"])
            dys = _st(net, dys)
            g[q + "sc.w"] = conv_wgrad(x, dys, p[q + "sc.w"].shape, b["stride"], 0)
            dx = _st(net, dx) + conv_dgrad(dys, _wq(net, p[q + "sc.w"]), b["stride"], 0, x.shape)
        else:
            dx = dx + d
        return _st(net, dx)
    if net.kind == "postbn":
        dy2, g[q + "bn2.g"], g[q + "bn2.b"] = bn_bwd(d, c["bn2"], p[q + "bn2.g"])
        dy2 = _st(net, dy2)
        g[q + "conv2.w"] = conv_wgrad(c["a1"], dy2, p[q + "conv2.w"].shape, 1, 1)
        da1 = _st(net, conv_dgrad(dy2, _wq(net, p[q + "conv2.w"]), 1, 1, c["a1"].shape))
        dz1 = relu_bwd(da1, c["z1"])
        dy1, g[q + "bn1.g"], g[q + "bn1.b"] = bn_bwd(dz1, c["bn1"], p[q + "bn1.g"])
        dy1 = _st(net, dy1)
        g[q + "conv1.w"] = conv_wgrad(x, dy1, p[q + "conv1.w"].shape, b["stride"], 1)
        dx = conv_dgrad(dy1, _wq(net, p[q + "conv1.w"]), b["stride"], 1, x.shape)
        if b["proj"]:
            dys, g[q + "bns.g"], g[q + "bns.b"] = bn_bwd(d, c["bns"], p[q + "bns.g"])
            dys = _st(net, dys)
            g[q + "sc.w"] = conv_wgrad(x, dys, p[q + "sc.w"].shape, b["stride"], 0)
            dx = _st(net, dx) + conv_dgrad(dys, _wq(net, p[q + "sc.w"]), b["stride"], 0, x.shape)
        else:
            dx = dx + d
        return _st(net, dx)
    # pre-activation form
    g[q + "conv2.w"] = conv_wgrad(c["a1"], d, p[q + "conv2.w"].shape, 1, 1)
    da1 = _st(net, conv_dgrad(d, _wq(net, p[q + "conv2.w"]), 1, 1, c["a1"].shape))
    dz1 = relu_bwd(da1, c["z1"])
    dy1, g[q + "bn2.g"], g[q + "bn2.b"] = bn_bwd(dz1, c["bn2"], p[q + "bn2.g"])
    dy1 = _st(net, dy1)
    g[q + "conv1.w"] = conv_wgrad(c["o"], dy1, p[q + "conv1.w"].shape, b["stride"], 1)
    do = _st(net, conv_dgrad(dy1, _wq(net, p[q + "conv1.w"]), b["stride"], 1, c["o"].shape))
    dx_direct = 0.0
    if b["proj"]:
        g[q + "sc.w"] = conv_wgrad(c["o"], d, p[q + "sc.w"].shape, b["stride"], 0)
        do = _st(net, do + conv_dgrad(d, _wq(net, p[q + "sc.w"]), b["stride"], 0, c["o"].shape))
    else:
        dx_direct = d
    dz0 = relu_bwd(do, c["z0"])
    dx, g[q + "bn1.g"], g[q + "bn1.b"] = bn_bwd(dz0, c["bn1"], p[q + "bn1.g"])
    return _st(net, dx + dx_direct)


def _head_fwd(net, p, x, cache):
    cache["head.x"] = x
    if net.kind == "preact":
        z, cache["head.bn"] = bn_fwd(x, p["head.bn.g"], p["head.bn.b"], net.eps)
        cache["head.z"] = z
        x = _st(net, relu(z))
    pooled = avgpool_fwd(x)
    cache["head.pooled"] = pooled
    return linear_fwd(pooled, p["head.fc.w"], p["head.fc.b"])


def _head_bwd(net, p, dlogits, cache, g):
    g["head.fc.w"] = dlogits.T @ cache["head.pooled"]
    g["head.fc.b"] = dlogits.sum(axis=0)
    d = _st(net, avgpool_bwd(dlogits @ p["head.fc.w"], cache["head.x"].shape))
    if net.kind == "preact":
        d = relu_bwd(d, cache["head.z"])
        d, g["head.bn.g"], g["head.bn.b"] = bn_bwd(d, cache["head.bn"], p["head.bn.g"])
        d = _st(net, d)
    return d


def module_forward(net, k, p, x_k, cache=None):
    """F_k(x_k): stem (k = 0), the module's residual blocks, head (k = K-1: returns logits)."""
    cache = {} if cache is None else cache
    x = np.asarray(x_k, dtype=F)
    if k == 0:
        x = _stem_fwd(net, p, x, cache)
    for i, bi in enumerate(net.module_blocks[k]):
        x = _block_fwd(net, bi, p, x, cache)
        # an interior module's final output goes straight into the local loss; every other block
        # output is kept as an activation tensor
        if not (i == len(net.module_blocks[k]) - 1 and k < net.K - 1 and net.post):
            x = _st(net, x)
    if k == net.K - 1:
        x = _head_fwd(net, p, x, cache)
    return x


def module_fwd_bwd(net, k, params_flat, x_k, x_next_or_labels, kappa, rho):
    """Forward of module k, its local loss, and the gradients of that loss with respect to the
    module's parameters and its input x_k (x_{k+1} and kappa held constant).

    Returns dict(loss, rnorm2, out, r, seed, grads (flat, blob order), dx (None for k = 0)).
    """
    p = net.unpack(k, params_flat)
    cache = {}
    out = module_forward(net, k, p, x_k, cache)
    res = dict(out=out)
    if k == net.K - 1:
        loss, seed = softmax_ce(out, np.asarray(x_next_or_labels))
        res.update(loss=loss, rnorm2=0.0, r=None, seed=seed)
    else:
        kap = None if kappa is None else np.asarray(kappa, dtype=F)
        loss, rn2, r, seed = local_loss(out, np.asarray(x_next_or_labels, dtype=F), kap, rho)
        res.update(loss=loss, rnorm2=rn2, r=_st(net, r), seed=seed)
        seed = _st(net, seed)
    g = {}
    d = seed
    if k == net.K - 1:
        d = _head_bwd(net, p, d, cache, g)
    for bi in reversed(net.module_blocks[k]):
        d = _block_bwd(net, bi, p, d, cache, g)
    if k == 0:
        d = _stem_bwd(net, p, d, cache, g)
    res["grads"] = net.pack(k, g)
    res["dx"] = d
    return res


# ----------------------------------------------------------------------------
# update  (Eq. Parallel-ResNet-Backpropagation; Eq. Parallel-ResNet-Multiplier-Update)
# ----------------------------------------------------------------------------
def sgd_update(params_flat, grads_flat, lr, momentum=0.0, weight_decay=0.0, velocity=None):
    """theta <- theta - lr * g   (plain SGD; optional weight decay and heavy-ball momentum)."""
    g = np.asarray(grads_flat, dtype=F) + weight_decay * np.asarray(params_flat, dtype=F)
    if momentum != 0.0:
        velocity = g if velocity is None else momentum * velocity + g
        g = velocity
    return np.asarray(params_flat, dtype=F) - lr * g, velocity


def kappa_update(kappa, r, kappa_step):
    """kappa <- kappa + c * (F_k(x_k) - x_{k+1}).  The paper's step is c = eta/(2 beta) = lr/rho;
    the method-of-multipliers step is c = rho (then the new kappa equals the terminal adjoint)."""
    return np.asarray(kappa, dtype=F) + kappa_step * r


# ----------------------------------------------------------------------------
# layer-serial forward, written separately from the module code (consistency check)
# ----------------------------------------------------------------------------
def forward_serial(net, module_params, images):
    """The undecomposed network X_0 = S(y), X_{l+1} = X_l + F(X_l, W_l), logits = T(X_L):
    one pass over all blocks with the per-module parameter blobs, no module structure."""
    named = {}
    for k in range(net.K):
        named.update(net.unpack(k, module_params[k]))
    eps = net.eps
    x = np.asarray(images, dtype=F)
    st = net.stem
    x = conv_fwd(x, named["stem.conv.w"], st["stride"], st["pad"])
    if net.post:
        x = relu(bn_fwd(x, named["stem.bn.g"], named["stem.bn.b"], eps)[0])
        if st["pool"]:
            x = maxpool_fwd(x)[0]
    for bi, b in enumerate(net.blocks):
        q = "block%d." % bi
        if net.kind == "bottleneck":
            t = relu(bn_fwd(conv_fwd(x, named[q + "conv1.w"], 1, 0), named[q + "bn1.g"], named[q + "bn1.b"], eps)[0])
            t = relu(bn_fwd(conv_fwd(t, named[q + "conv2.w"], b["stride"], 1), named[q + "bn2.g"], named[q + "bn2.b"], eps)[0])
            t = bn_fwd(conv_fwd(t, named[q + "conv3.w"], 1, 0), named[q + "bn3.g"], named[q + "bn3.b"], eps)[0]
            s = (bn_fwd(conv_fwd(x, named[q + "sc.w"], b["stride"], 0), named[q + "bns.g"], named[q + "bns.b"], eps)[0]
                 if b["proj"] else x)
            x = s + t
        elif net.kind == "postbn":
            t = conv_fwd(x, named[q + "conv1.w"], b["stride"], 1)
            t = relu(bn_fwd(t, named[q + "bn1.g"], named[q + "bn1.b"], eps)[0])
            t = conv_fwd(t, named[q + "conv2.w"], 1, 1)
            t = bn_fwd(t, named[q + "bn2.g"], named[q + "bn2.b"], eps)[0]
            if b["proj"]:
                s = bn_fwd(conv_fwd(x, named[q + "sc.w"], b["stride"], 0),
                           named[q + "bns.g"], named[q + "bns.b"], eps)[0]
            else:
                s = x
            x = s + t
        else:
            o = relu(bn_fwd(x, named[q + "bn1.g"], named[q + "bn1.b"], eps)[0])
            t = conv_fwd(o, named[q + "conv1.w"], b["stride"], 1)
            t = relu(bn_fwd(t, named[q + "bn2.g"], named[q + "bn2.b"], eps)[0])
            t = conv_fwd(t, named[q + "conv2.w"], 1, 1)
            s = conv_fwd(o, named[q + "sc.w"], b["stride"], 0) if b["proj"] else x
            x = s + t
    if net.kind == "preact":
        x = relu(bn_fwd(x, named["head.bn.g"], named["head.bn.b"], eps)[0])
    return linear_fwd(avgpool_fwd(x), named["head.fc.w"], named["head.fc.b"])


# ----------------------------------------------------------------------------
# one whole layer-parallel step (Algorithm 1 without the AuxNet distillation)
# ----------------------------------------------------------------------------
def layer_parallel_step(net, module_params, aux_params, images, labels, kappas, rho, lr,
                        kappa_step=None, post=None):
    """AuxNet chain, K independent module forward+backward passes, SGD and multiplier updates.
    ``kappas``: list of K-1 arrays or None (penalty method).  Returns the new parameters, new
    multipliers and the per-module results."""
    xs = [np.asarray(images, dtype=F)] + auxnet_forward(net, aux_params, images, post=post)
    results, new_params, new_kappas = [], [], []
    for k in range(net.K):
        last = k == net.K - 1
        tgt = labels if last else xs[k + 1]
        kap = None if (kappas is None or last) else kappas[k]
        res = module_fwd_bwd(net, k, module_params[k], xs[k], tgt, kap, rho)
        results.append(res)
        new_params.append(sgd_update(module_params[k], res["grads"], lr)[0])
        if kap is not None:
            c = rho if kappa_step is None else kappa_step
            new_kappas.append(kappa_update(kap, res["r"], c))
    return new_params, (new_kappas if kappas is not None else None), results, xs
