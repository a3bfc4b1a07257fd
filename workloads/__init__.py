"""Workload descriptions and seeded synthetic inputs.

This package is the only code shared by the CPU oracle's tests and the CUDA
path's tests: it names the five workloads (network shapes, batch sizes, loss
settings) and draws every random tensor from one counter-based generator.  It
contains none of the method's arithmetic: no convolution, no normalisation,
no loss.
"""
from .configs import CONFIGS, get_config, scaled, with_modules  # noqa: F401
from .gen import (normal, uniform_int, make_images, make_labels, make_params,  # noqa: F401
                  make_kappa, round_bf16, augment_crop_flip)
