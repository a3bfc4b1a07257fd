"""CPU-side checks of the C ABI: the library loads, exports every declared symbol, and its host
logic (descriptor validation, parameter layouts, boundary shapes, workspace sizing) agrees with the
oracle's independently written network description."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2112_05387_b200 as lp
from conftest import small_cfg
from oracle import lp_oracle as O
from workloads import CONFIGS, get_config

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    import __graft_entry__ as g
    g.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "lp.h")).read()
    declared = set(re.findall(r"\b(lp_[a-z0-9_]+)\s*\(", header))
    declared -= {"lp_net_desc", "lp_param_entry", "lp_handle", "lp_status"}
    lib = ctypes.CDLL(lp.library_path())
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert declared == set(lp.EXPORTED_SYMBOLS)


@pytest.mark.parametrize("name", list(CONFIGS))
def test_layouts_and_boundaries_match_oracle(name):
    cfg = get_config(name)
    net = O.Net(cfg)
    desc = lp.desc_from_config(cfg)
    assert lp.lp_validate_desc(desc) == 0
    for k in range(net.K):
        assert lp.lp_param_layout(desc, k) == [(n, kd, tuple(s)) for n, kd, s in net.param_layout(k)]
        assert lp.lp_boundary_shape_desc(desc, k) == tuple(net.boundary[k])
    for k in range(net.K - 1):
        assert lp.lp_param_layout(desc, lp.LP_AUX(k)) == [(n, kd, tuple(s)) for n, kd, s in net.param_layout(O.LP_AUX(k))]
    assert lp.lp_workspace_bytes(desc) > 0


def test_custom_configs_layouts():
    for cfg in (small_cfg("postbn"), small_cfg("preact"),
                small_cfg("postbn", stem="conv7x7s2_maxpool", H=16, W=16, stage_channels=(8, 8), stage_stride=(1, 1))):
        net = O.Net(cfg)
        desc = lp.desc_from_config(cfg)
        for k in range(net.K):
            assert lp.lp_param_layout(desc, k) == [(n, kd, tuple(s)) for n, kd, s in net.param_layout(k)]


def test_parameter_counts_of_named_networks():
    # ResNet-110 has about 1.7 million parameters (paper, Section 5)
    cfg = get_config("resnet110")
    net = O.Net(cfg)
    total = sum(net.param_count(k) for k in range(net.K))
    assert 1.6e6 < total < 1.8e6
    # ResNet-50 (bottleneck blocks, projection shortcuts with BN, 1000 classes): the textbook 25,557,032
    cfg = get_config("resnet50")
    net = O.Net(cfg)
    assert sum(net.param_count(k) for k in range(net.K)) == 25557032
    desc = lp.desc_from_config(cfg)
    assert sum(int(np.prod(s)) for k in range(net.K) for _, _, s in lp.lp_param_layout(desc, k)) == 25557032


def test_bad_descriptors_are_rejected():
    good = lp.desc_from_config(get_config("tiny"))
    assert lp.lp_validate_desc(good) == 0
    for field, value in [("struct_size", 12), ("dtype", 7), ("N", 0), ("K", 0), ("K", 17), ("post_add_relu", 1),
                         ("num_stages", 0), ("bn_eps", 0.0), ("aux_convs_per_boundary", 3), ("stem_channels", 6)]:
        d = lp.desc_from_config(get_config("tiny"))
        setattr(d, field, value)
        assert lp.lp_validate_desc(d) != 0, field
        assert lp.lp_workspace_bytes(d) == 0
    d = lp.desc_from_config(get_config("tiny"))
    d.module_block_end[1] = 5
    assert lp.lp_validate_desc(d) != 0
    d = lp.desc_from_config(get_config("tiny"))
    d.stage_stride[0] = 3
    assert lp.lp_validate_desc(d) != 0
    assert "null" in lp.lp_status_string(-1)
    with pytest.raises(lp.LpError):
        lp.lp_param_layout(good, 9)


def test_with_modules_splits_the_blocks_evenly_and_validates():
    """Re-splitting a workload into K modules (the K sweep of the speed-up accounting) keeps the
    network and yields descriptors the library accepts; K = 1 is the layer-serial network."""
    import paper_2112_05387_b200 as lp
    from workloads import with_modules
    for name, total in (("wrn28_10", 12), ("resnet110", 54), ("tiny", 2)):
        for K in (1, 2, 3, 4, 6):
            if K > total:
                with pytest.raises(ValueError):
                    with_modules(name, K)
                continue
            cfg = with_modules(name, K)
            ends = cfg["module_block_end"]
            assert len(ends) == K == cfg["K"] and ends[-1] == total and ends == sorted(set(ends))
            sizes = np.diff([0] + ends)
            assert sizes.max() - sizes.min() <= 1
            assert lp.lp_validate_desc(lp.desc_from_config(cfg)) == 0
            assert O.Net(cfg).K == K


def test_recursive_auxnet_layouts_match_the_oracle():
    """aux_recursive = 1: LP_REAUX(k, j) has the layout of AuxNet_j; indices past the last stack are refused."""
    import paper_2112_05387_b200 as lp
    from conftest import small_cfg
    from oracle import lp_oracle as O
    cfg = small_cfg("preact", stage_channels=(8, 16), stage_blocks=(2, 2), module_block_end=(1, 2, 3, 4), N=3)
    net = O.Net(cfg)
    desc = lp.desc_from_config(cfg, aux_recursive=True)
    assert lp.lp_validate_desc(desc) == 0
    assert lp.lp_workspace_bytes(desc) > lp.lp_workspace_bytes(lp.desc_from_config(cfg))
    for k in range(1, net.K):
        for j in range(k):
            lay = lp.lp_param_layout(desc, lp.LP_REAUX(k, j))
            assert [(n, tuple(s)) for n, _, s in lay] == [(n, tuple(s)) for n, _, s in net.param_layout(O.LP_AUX(j))]
    with pytest.raises(lp.LpError):
        lp.lp_param_layout(desc, lp.LP_REAUX(net.K, 0))
    desc.aux_recursive = 2
    assert lp.lp_validate_desc(desc) != 0
