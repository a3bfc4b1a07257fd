"""The five workloads: a tiny fp32 network plus four CIFAR/ImageNet-shaped ones.

Each entry is a plain dict whose keys mirror the fields of ``lp_net_desc``
(include/lp.h) plus the loss settings and seeds of the workload.  The shapes
stand in for CIFAR-10/100 and ImageNet batches: only image size, class count
and batch size are taken from those datasets, the pixels are synthetic.

Keys
----
dtype            "f32" | "bf16": storage type of activations on the GPU path
N,H,W,C_in       input batch (NHWC)
num_classes
stem_kind        "conv3x3" | "conv7x7s2_maxpool"
stem_channels
block_kind       "postbn" (conv-BN-ReLU-conv-BN + shortcut), "bottleneck" (1x1-3x3-1x1, inner width C_out/4)
                 | "preact" (BN-ReLU-conv-BN-ReLU-conv + shortcut)
stage_channels / stage_blocks / stage_stride
module_block_end cumulative block index that ends each of the K modules
aux_convs        3x3 convolutions per AuxNet boundary (1 or 2)
aux_width_div    hidden width of a 2-conv AuxNet = C_out / aux_width_div
loss             "penalty" | "al"; rho; kappa_std (std of the initial multiplier)
"""
import copy

_COMMON = dict(bn_eps=1e-5, seed=0, lr=0.1)

CONFIGS = {
    # configs[0]: tiny fp32 network, the 1e-4 parity case.
    "tiny": dict(
        dtype="f32", N=8, H=8, W=8, C_in=3, num_classes=10,
        stem_kind="conv3x3", stem_channels=8, block_kind="postbn",
        stage_channels=[8], stage_blocks=[2], stage_stride=[1],
        module_block_end=[1, 2], aux_convs=1, aux_width_div=1,
        loss="al", rho=1.0, kappa_std=0.1, augment=False, **_COMMON),
    # configs[1]: ResNet-56, K=3 at the stage boundaries, penalty loss.
    "resnet56": dict(
        dtype="bf16", N=128, H=32, W=32, C_in=3, num_classes=10,
        stem_kind="conv3x3", stem_channels=16, block_kind="postbn",
        stage_channels=[16, 32, 64], stage_blocks=[9, 9, 9], stage_stride=[1, 2, 2],
        module_block_end=[9, 18, 27], aux_convs=2, aux_width_div=1,
        loss="penalty", rho=1.0, kappa_std=0.0, augment=True, **_COMMON),
    # configs[2]: ResNet-110, K=6 modules of 9 blocks, augmented Lagrangian.
    "resnet110": dict(
        dtype="bf16", N=128, H=32, W=32, C_in=3, num_classes=100,
        stem_kind="conv3x3", stem_channels=16, block_kind="postbn",
        stage_channels=[16, 32, 64], stage_blocks=[18, 18, 18], stage_stride=[1, 2, 2],
        module_block_end=[9, 18, 27, 36, 45, 54], aux_convs=2, aux_width_div=1,
        loss="al", rho=1.0, kappa_std=0.0, augment=False, **_COMMON),
    # configs[3]: WideResNet-28-10, pre-activation, K=4 modules of 3 blocks.
    "wrn28_10": dict(
        dtype="bf16", N=128, H=32, W=32, C_in=3, num_classes=10,
        stem_kind="conv3x3", stem_channels=16, block_kind="preact",
        stage_channels=[160, 320, 640], stage_blocks=[4, 4, 4], stage_stride=[1, 2, 2],
        module_block_end=[3, 6, 9, 12], aux_convs=2, aux_width_div=4,
        loss="penalty", rho=0.5, kappa_std=0.0, augment=False, **_COMMON),
    # configs[4]: ImageNet-shaped ResNet-34, K=4 at the stage boundaries, AL.
    "resnet34": dict(
        dtype="bf16", N=64, H=224, W=224, C_in=3, num_classes=1000,
        stem_kind="conv7x7s2_maxpool", stem_channels=64, block_kind="postbn",
        stage_channels=[64, 128, 256, 512], stage_blocks=[3, 4, 6, 3],
        stage_stride=[1, 2, 2, 2], module_block_end=[3, 7, 13, 16],
        aux_convs=2, aux_width_div=4,
        loss="al", rho=1.0, kappa_std=0.0, augment=False, **_COMMON),
    # beyond the five named configurations: ImageNet-shaped ResNet-50 (bottleneck blocks), the network of
    # the paper's ImageNet experiment; K=4 at the stage boundaries, penalty loss.
    "resnet50": dict(
        dtype="bf16", N=32, H=224, W=224, C_in=3, num_classes=1000,
        stem_kind="conv7x7s2_maxpool", stem_channels=64, block_kind="bottleneck",
        stage_channels=[256, 512, 1024, 2048], stage_blocks=[3, 4, 6, 3],
        stage_stride=[1, 2, 2, 2], module_block_end=[3, 7, 13, 16],
        aux_convs=2, aux_width_div=4,
        loss="penalty", rho=1.0, kappa_std=0.0, augment=False, **_COMMON),
}


def get_config(name):
    cfg = copy.deepcopy(CONFIGS[name])
    cfg["name"] = name
    cfg["K"] = len(cfg["module_block_end"])
    return cfg


def scaled(name, N=None, H=None, W=None, dtype=None):
    """A workload with a smaller batch or image, same network: parity-test sizes."""
    cfg = get_config(name)
    if N is not None:
        cfg["N"] = N
    if H is not None:
        cfg["H"] = H
    if W is not None:
        cfg["W"] = W
    if dtype is not None:
        cfg["dtype"] = dtype
    return cfg


def with_modules(name, K, **kw):
    """The workload `name` re-split into K modules of (nearly) equal block count; K = 1 is the
    layer-serial network (no auxiliary variables).  Extra keywords go to `scaled`."""
    cfg = scaled(name, **kw)
    total = sum(cfg["stage_blocks"])
    if not 1 <= K <= total:
        raise ValueError("K must be in 1..%d" % total)
    cfg["module_block_end"] = [(total * (k + 1)) // K for k in range(K)]
    cfg["K"] = K
    return cfg
