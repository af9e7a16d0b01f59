"""Host-side checks that need no GPU: the library builds, loads, exports every declared symbol,
and rejects bad configurations before touching CUDA."""
import ctypes
import os
import re
from dataclasses import replace

import pytest

import emc2_gen as gen

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def pkg():
    import paper_2507_04123_b200 as p
    from paper_2507_04123_b200 import build
    build.build()
    return p


def test_library_exports_every_declared_symbol(pkg):
    lib = pkg.load_library()
    header = open(os.path.join(ROOT, "include", "emc2_bridge.h")).read()
    declared = set(re.findall(r"\b(emc2_[a-z_0-9]+)\s*\(", header))
    assert declared == set(pkg.ABI_SYMBOLS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_config_struct_layout_matches_the_header(pkg):
    # 4 ints, 2 grids of (3f, 3f, 3i, i), 7 ints, float, int, 7 floats, int, 16 bytes, float
    assert ctypes.sizeof(pkg.Emc2Grid) == 40
    assert ctypes.sizeof(pkg.Emc2Config) == 16 + 80 + 28 + 4 + 4 + 28 + 4 + 16 + 4


def test_status_strings(pkg):
    lib = pkg.load_library()
    texts = {lib.emc2_status_string(s).decode() for s in range(0, -7, -1)}
    assert len(texts) == 7 and "ok" in texts
    assert lib.emc2_bridge_kernel_kinds() == len({lib.emc2_bridge_kernel_name(k) for k in range(lib.emc2_bridge_kernel_kinds())})


def _create(pkg, cfg):
    h = ctypes.c_void_p()
    rc = pkg.load_library().emc2_bridge_create(ctypes.byref(cfg), ctypes.byref(h))
    if rc == 0:
        pkg.load_library().emc2_bridge_destroy(h)
    return rc


def test_bad_configurations_are_rejected_on_the_host(pkg):
    w = gen.TINY
    BAD = pkg.bridge.EMC2_ERR_BAD_CONFIG
    good = pkg.config_from_workload(w)
    assert _create(pkg, good) in (0, pkg.bridge.EMC2_ERR_CUDA)        # no GPU here: CUDA error, not a fallback

    def mutated(**kw):
        return pkg.config_from_workload(replace(w, **kw))

    zero_voxel = replace(w.grids[0], voxel=(0.0, 0.05, 0.1))
    assert _create(pkg, mutated(grids=(zero_voxel, w.grids[1]))) == BAD
    huge = replace(w.grids[0], dims=(1 << 12, 1 << 12, 1 << 9))
    assert _create(pkg, mutated(grids=(huge, w.grids[1]))) == BAD              # >= 2^32 cells
    capped_fine = replace(w.grids[0], max_points=8)                             # a cap is fine on any grid
    assert _create(pkg, mutated(grids=(capped_fine, w.grids[1]))) in (0, pkg.bridge.EMC2_ERR_CUDA)
    tall_pillars = replace(w.grids[1], dims=(440, 500, 2))
    assert _create(pkg, mutated(grids=(w.grids[0], tall_pillars))) == BAD
    assert _create(pkg, mutated(feat_c=62)) == BAD
    assert _create(pkg, mutated(feat_stride=3)) == BAD
    cfg = pkg.config_from_workload(w)
    cfg.feat_stride = 2                                                        # map too small for the image
    assert _create(pkg, cfg) == BAD
    assert _create(pkg, mutated(thresholds=(40.0, 20.0))) == BAD
    assert _create(pkg, mutated(num_experts=3)) == BAD                         # lut names expert 3
    assert _create(pkg, mutated(num_experts=17)) == BAD
    assert _create(pkg, mutated(C=6)) == BAD
    cfg = pkg.config_from_workload(w)
    cfg.max_batch = 33
    assert _create(pkg, cfg) == BAD
    cfg = pkg.config_from_workload(w)
    cfg.num_cameras = 9
    assert _create(pkg, cfg) == BAD
    lib = pkg.load_library()
    assert lib.emc2_bridge_create(None, None) == pkg.bridge.EMC2_ERR_INVALID_ARG
    assert lib.emc2_bridge_destroy(None) == 0
    assert lib.emc2_bridge_status(None, None) == pkg.bridge.EMC2_ERR_INVALID_ARG


def test_binding_refuses_to_run_without_cuda(pkg):
    import torch
    if torch.cuda.is_available():
        pytest.skip("CUDA present")
    with pytest.raises(RuntimeError):
        pkg.Bridge(pkg.config_from_workload(gen.TINY))


def test_tuning_and_timeline_reject_a_null_handle(pkg):
    lib = pkg.load_library()
    assert lib.emc2_bridge_set_tuning(None, 0, 0) == pkg.bridge.EMC2_ERR_INVALID_ARG
    assert lib.emc2_bridge_profile_timeline(None, None, None, None, 0) == pkg.bridge.EMC2_ERR_INVALID_ARG
    assert set(pkg.bridge.TUNE_NAMES.values()) == set(range(len(pkg.bridge.TUNE_NAMES)))
