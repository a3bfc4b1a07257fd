"""Seeded synthetic inputs from one counter-based generator.

Every tensor is a pure function of (seed, stream name, element index): the
64-bit counter ``key(seed, name) + (i+1)*GOLDEN`` is passed through the
splitmix64 finaliser, pairs of 53-bit uniforms go through the Box-Muller
transform.  Nothing here depends on draw order, so the oracle's tests and the
CUDA tests receive identical values whatever order they ask in.
"""
import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z):
    z = z.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        z ^= z >> np.uint64(30)
        z *= _M1
        z ^= z >> np.uint64(27)
        z *= _M2
        z ^= z >> np.uint64(31)
    return z


def _key(seed, name):
    h = np.uint64(0xCBF29CE484222325)          # FNV-1a over the stream name
    with np.errstate(over="ignore"):
        for b in name.encode():
            h = (h ^ np.uint64(b)) * np.uint64(0x100000001B3)
        h = h ^ (np.uint64(seed) * _GOLDEN)
    return _mix(np.array([h], dtype=np.uint64))[0]


def _u64(seed, name, count, offset=0):
    idx = np.arange(offset + 1, offset + count + 1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _mix(_key(seed, name) + idx * _GOLDEN)


def _uniform01(seed, name, count, offset=0):
    """Uniform on (0,1): 53 bits, shifted by half an ulp so 0 is never returned."""
    bits = _u64(seed, name, count, offset) >> np.uint64(11)
    return (bits.astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed, name, shape, std=1.0, mean=0.0):
    n = int(np.prod(shape))
    u = _uniform01(seed, name, 2 * n)
    z = np.sqrt(-2.0 * np.log(u[0::2])) * np.cos(2.0 * np.pi * u[1::2])
    return (mean + std * z).reshape(shape)


def uniform_int(seed, name, shape, high):
    n = int(np.prod(shape))
    return (_u64(seed, name, n) % np.uint64(high)).astype(np.int32).reshape(shape)


def round_bf16(a):
    """Round float values to the nearest bfloat16 (ties to even); returns float32."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    out = ((u + r) & np.uint32(0xFFFF0000)).view(np.float32)
    return out.reshape(f.shape)


def storage_round(a, dtype):
    return round_bf16(a) if dtype == "bf16" else np.ascontiguousarray(a, dtype=np.float32)


def augment_crop_flip(seed, images, pad=4):
    """Zero-pad by ``pad``, take a random crop of the original size, flip with p = 1/2."""
    n, h, w, c = images.shape
    padded = np.zeros((n, h + 2 * pad, w + 2 * pad, c), dtype=images.dtype)
    padded[:, pad:pad + h, pad:pad + w, :] = images
    oy = uniform_int(seed, "aug/oy", (n,), 2 * pad + 1)
    ox = uniform_int(seed, "aug/ox", (n,), 2 * pad + 1)
    fl = uniform_int(seed, "aug/flip", (n,), 2)
    out = np.empty_like(images)
    for i in range(n):
        crop = padded[i, oy[i]:oy[i] + h, ox[i]:ox[i] + w, :]
        out[i] = crop[:, ::-1, :] if fl[i] else crop
    return out


def make_images(cfg, seed=None):
    seed = cfg["seed"] + 1 if seed is None else seed
    x = normal(seed, "images", (cfg["N"], cfg["H"], cfg["W"], cfg["C_in"]))
    if cfg.get("augment"):
        x = augment_crop_flip(seed + 1, x)
    return storage_round(x, cfg["dtype"])


def make_labels(cfg, seed=None):
    seed = cfg["seed"] + 1 if seed is None else seed
    return uniform_int(seed, "labels", (cfg["N"],), cfg["num_classes"])


def make_kappa(cfg, k, shape, seed=None, std=None):
    """Multiplier attached to the constraint F_k(x_k) = x_{k+1}."""
    seed = cfg["seed"] if seed is None else seed
    std = cfg["kappa_std"] if std is None else std
    if std == 0.0:
        return np.zeros(shape, dtype=np.float32)
    return storage_round(normal(seed, "kappa/%d" % k, shape, std=std), cfg["dtype"])


def make_params(layout, seed, tag, perturb_bn=False, dtype="f32"):
    """Fill a parameter layout: a list of (name, kind, shape) in blob order.

    conv_w / fc_w ~ N(0, 2/fan_in) (fan_in = product of all dims but the first),
    bn_gamma = 1, bn_beta = 0, fc_b = 0.  With ``perturb_bn`` the affine
    parameters and the bias get N(., 0.1^2) noise so that tests can tell them
    apart.  Values are rounded to the storage type so that a bf16 copy of the
    fp32 master is exact at the first step.
    """
    parts = []
    for name, kind, shape in layout:
        shape = tuple(int(s) for s in shape if int(s) > 0)
        n = int(np.prod(shape))
        stream = "%s/%s" % (tag, name)
        if kind in ("conv_w", "fc_w"):
            fan_in = n // shape[0]
            v = normal(seed, stream, (n,), std=np.sqrt(2.0 / fan_in))
        elif kind == "bn_gamma":
            v = np.ones(n) if not perturb_bn else normal(seed, stream, (n,), std=0.1, mean=1.0)
        elif kind in ("bn_beta", "fc_b"):
            v = np.zeros(n) if not perturb_bn else normal(seed, stream, (n,), std=0.1)
        else:
            raise ValueError(kind)
        parts.append(storage_round(v, dtype).astype(np.float32))
    return np.concatenate(parts) if parts else np.zeros(0, dtype=np.float32)
