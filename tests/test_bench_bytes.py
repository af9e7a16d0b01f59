"""The byte counts behind bench.py's bandwidth figures, re-derived by hand for one small case."""
import torch

import bench
import emc2_gen as gen


def test_algorithmic_bytes_of_the_tiny_workload():
    w = gen.TINY                      # 1 frame, 16,384 points of 4 floats, 1 camera, 64 channels, 3 + 1 experts
    B, N, m0, m1, texels = 1, 16384, 9000, 4000, 1234
    assert (w.C, w.feat_c, w.K) == (4, 64, 1)
    E = w.num_experts
    gy, gx = w.grids[1].dims[1], w.grids[1].dims[0]
    # stage 1: points read; point_voxel of two scales written; per voxel coords (16) + count (4) + mean (16);
    # the BEV image of C planes
    vox = N * 16 + N * 2 * 4 + (m0 + m1) * (16 + 4 + 16) + 4 * gy * gx * 4
    # stage 2: points and matrices read, each distinct texel row read once; uvd (12), mask (1), camera (1)
    # and the feature row (256) written
    pg = N * 16 + 48 + texels * 256 + N * (12 + 1 + 1 + 256)
    # stages 3 - 4: points, mask and rows read; expert (1), permutation (4), point row and feature row written;
    # offsets
    rd = N * (16 + 1 + 256) + N * (1 + 4 + 16 + 256) + (E + 1) * 4
    got = bench.algorithmic_bytes(w, B, N, m0, m1, texels)
    assert got == {"voxelize": vox, "project_gather": pg, "route_dispatch": rd, "total": vox + pg + rd}
    kb = bench.kernel_bytes(w, B, N, texels)
    assert kb["project_gather"] == pg
    assert kb["dispatch_scatter"] == N * (1 + 16 + 256) + N * (4 + 16 + 256)
    # one pass over the rows: points, uvd, camera, expert and texels read; permutation, point row and the
    # feature row at both of its places written
    assert kb["gather_scatter"] == N * (16 + 12 + 1 + 1) + texels * 256 + N * (4 + 16 + 2 * 256)
    one = bench.one_call_bytes(w, B, N, m0, m1, texels)
    assert one == vox + (N * 16 + 48 + N * (12 + 1 + 1 + 1)) + kb["gather_scatter"] + (E + 1) * 4
    assert one < got["total"]


def test_distinct_texels_counts_shared_taps_once():
    w = gen.TINY                      # stride 4: pixels 0..3 share texel column 0
    uvd = torch.tensor([[[1.0, 1.0, 5.0], [2.0, 2.0, 5.0], [9.0, 1.0, 5.0], [0.0, 0.0, 5.0]]])
    cam = torch.tensor([[0, 0, 0, -1]], dtype=torch.int8)
    # points 0 and 1 use texels (0..1, 0..1); point 2 uses (2..3, 0..1); the last point sees no camera
    assert bench.distinct_texels(w, {"uvd": uvd, "cam": cam}) == 8


def test_every_bandwidth_figure_pairs_a_time_with_the_bytes_that_path_moves():
    # 1,000 MB in 0.25 ms is 4,000 GB/s: half of 8 TB/s.  The staged count (1,400 MB) only counts against the
    # staged time; over the one-call time it appears under a name that says so and is not the headline.
    f = bench.bridge_fractions(own_bytes=1_000_000_000, staged_bytes=1_400_000_000, ms_step=0.25, staged_ms=0.4,
                               peak=6500.0, peak_kind="measured")
    assert f["one_call_bytes_per_step"] == 1_000_000_000
    assert abs(f["bridge_own_gbs"] - 4000.0) < 1e-6
    assert abs(f["bridge_frac_of_8tbs_own_bytes"] - 0.5) < 1e-12 and f["target_50pct_of_8tbs_met"] is True
    assert abs(f["bridge_frac_of_measured_copy_own_bytes"] - 4000.0 / 6500.0) < 1e-12
    assert abs(f["staged_path"]["gbs"] - 3500.0) < 1e-6 and abs(f["staged_path"]["frac_of_8tbs"] - 0.4375) < 1e-12
    assert abs(f["equivalent_staged_bandwidth"]["frac_of_8tbs"] - 0.7) < 1e-12
    assert "bridge_frac_of_8tbs" not in f and "bridge_gbs" not in f        # the ambiguous names are gone
    slower = bench.bridge_fractions(1_000_000_000, 1_400_000_000, 0.26, 0.4, 6500.0, "measured")
    assert slower["target_50pct_of_8tbs_met"] is False
