"""emc2_route_dispatch_static, the dispatch entry point for hosts that must not allocate.

Some users of the library run where device allocation is off limits at dispatch time: inside an
engine that owns the device heap, or in a real-time loop that may not wait on the driver's
allocator.  For them the library keeps one small scratch array inside its own image and offers
stages 3 and 4 without a handle.  The GPU test drives that entry point through the C ABI twice
in a row, on different shapes, and requires the same results as the handle-based
emc2_route_dispatch and as the CPU oracle's routing and dispatch of the same inputs: integers
identical, rows identical bit for bit (they are copies).  The file
name sorts last so that a run stopping at the first failure has already run everything else.
"""
import ctypes

import numpy as np
import pytest
import torch

import emc2_gen as gen


def _pkg():
    import paper_2507_04123_b200 as pkg
    from paper_2507_04123_b200 import build
    build.build()
    return pkg


def test_oversized_call_is_refused_before_any_cuda_work():
    pkg = _pkg()
    lib = pkg.load_library()
    cfg = pkg.config_from_workload(gen.KITTI)
    tiles = pkg.bridge.STATIC_SCRATCH_ENTRIES // (cfg.num_experts * 32) + 1
    rc = lib.emc2_route_dispatch_static(ctypes.byref(cfg), 32, tiles * 256, *([None] * 9))
    assert rc == pkg.bridge.EMC2_ERR_TOO_LARGE
    assert b"scratch" in lib.emc2_status_string(rc)
    # a frame length near INT_MAX must not wrap the tile count around to something that fits
    assert lib.emc2_route_dispatch_static(ctypes.byref(cfg), 1, 2**31 - 1, *([None] * 9)) == pkg.bridge.EMC2_ERR_TOO_LARGE
    cfg.num_experts = 3                                    # lut names expert 3
    assert lib.emc2_route_dispatch_static(ctypes.byref(cfg), 1, 256, *([None] * 9)) == pkg.bridge.EMC2_ERR_BAD_CONFIG
    assert lib.emc2_route_dispatch_static(None, 1, 256, *([None] * 9)) == pkg.bridge.EMC2_ERR_INVALID_ARG


def test_binding_refuses_tensors_that_are_not_on_the_configured_device():
    pkg = _pkg()
    cfg = pkg.config_from_workload(gen.KITTI)
    cpu = torch.zeros((1, 4, 4))
    with pytest.raises(ValueError, match="device"):
        pkg.route_dispatch_static(cfg, cpu, cpu, cpu, {})


@pytest.mark.gpu
def test_static_scratch_dispatch_matches_the_handle_based_call_twice_in_a_row(oracle):
    pkg = _pkg()
    assert torch.cuda.is_available()
    # Two calls back to back, the second smaller and with another row width, so that entries the
    # first call left in the shared scratch would show up if the second relied on them.
    for w in (gen.NUSCENES.with_shape(3, 40_001), gen.KITTI.with_shape(2, 9_000)):
        cfg = pkg.config_from_workload(w)
        batch = gen.make_batch(w, feature_frames=1)
        d = {k: torch.from_numpy(v).cuda() for k, v in batch.items()}
        br = pkg.Bridge(cfg)
        pg = br.project_gather(d["points"], d["proj"], d["feat"])
        want = br.route_dispatch(d["points"], pg["vis_mask"], pg["gathered"])
        br.status()
        got = {k: torch.full_like(v, 0x55) if v.dtype != torch.float32 else torch.full_like(v, float("nan"))
               for k, v in want.items()}
        pkg.route_dispatch_static(cfg, d["points"], pg["vis_mask"], pg["gathered"], got)
        torch.cuda.synchronize()
        for k in ("expert", "offsets", "perm"):
            assert torch.equal(got[k], want[k]), k
        for k in ("points_out", "feat_out"):
            assert np.array_equal(got[k].cpu().numpy().view(np.uint32), want[k].cpu().numpy().view(np.uint32)), k
        assert len(torch.unique(want["expert"])) > 1
        # and against the oracle, so that a fault shared by both CUDA entry points cannot hide
        pts, vis, rows = batch["points"], pg["vis_mask"].cpu().numpy(), pg["gathered"].cpu().numpy()
        ref_expert = oracle.route(pts, vis, w.thresholds, w.lut)
        ref_offsets, ref_perm, ref_points, ref_rows = oracle.dispatch(ref_expert, pts, rows, w.num_experts)
        assert np.array_equal(got["expert"].cpu().numpy(), ref_expert)
        assert np.array_equal(got["offsets"].cpu().numpy(), ref_offsets)
        assert np.array_equal(got["perm"].cpu().numpy(), ref_perm)
        assert np.array_equal(got["points_out"].cpu().numpy().view(np.uint32), ref_points.view(np.uint32))
        assert np.array_equal(got["feat_out"].cpu().numpy().view(np.uint32), ref_rows.view(np.uint32))
        br.close()
