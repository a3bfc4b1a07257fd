import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu)")


def small_cfg(kind="postbn", stem="conv3x3", N=4, H=8, W=8, K=2, dtype="f32", classes=5,
              stage_channels=(8, 16), stage_blocks=(1, 1), stage_stride=(1, 2),
              module_block_end=(1, 2), aux_convs=2, aux_width_div=2, stem_channels=8, C_in=3):
    """A small custom workload used by the oracle tests (covers stride-2 projection blocks)."""
    cfg = dict(name="small-%s" % kind, dtype=dtype, N=N, H=H, W=W, C_in=C_in, num_classes=classes,
               stem_kind=stem, stem_channels=stem_channels, block_kind=kind,
               stage_channels=list(stage_channels), stage_blocks=list(stage_blocks),
               stage_stride=list(stage_stride), module_block_end=list(module_block_end),
               aux_convs=aux_convs, aux_width_div=aux_width_div, loss="al", rho=0.7,
               kappa_std=0.1, augment=False, bn_eps=1e-5, seed=0, lr=0.1)
    cfg["K"] = len(cfg["module_block_end"])
    return cfg


@pytest.fixture
def make_small_cfg():
    return small_cfg
