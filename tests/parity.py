"""Shared comparison helpers for the GPU-vs-oracle parity tests."""
import numpy as np
import torch

ATOL, RTOL = 1e-4, 1e-5          # |a - b| <= 1e-4 + 1e-5 * |b| for every float output


def close(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    err = np.abs(a - b)
    bad = err > ATOL + RTOL * np.abs(b)
    return not bad.any(), float(err.max(initial=0.0)), int(bad.sum())


def to_dev(batch, device="cuda"):
    return {k: torch.from_numpy(v).to(device) for k, v in batch.items()}


def np_(t):
    return t.detach().cpu().numpy()


def compare_bridge(w, ref, bufs, check_bev=True):
    """Asserts every output of the three stage calls against the oracle's dictionary."""
    vox, pg, rd = bufs["vox"], bufs["pg"], bufs["rd"]
    nv = np_(vox["num_voxels"])
    for s in range(2):
        r = ref[f"vox{s}"]
        M = r["num_voxels"]
        assert nv[s] == M, f"scale {s}: {nv[s]} voxels, oracle {M}"
        assert np.array_equal(np_(vox["coords"][s])[:M], r["coords"]), f"coords scale {s}"
        assert np.array_equal(np_(vox["counts"][s])[:M], r["counts"]), f"counts scale {s}"
        assert np.array_equal(np_(vox["point_voxel"][s]), r["point_voxel"]), f"point_voxel scale {s}"
        ok, mx, nbad = close(np_(vox["mean"][s])[:M], r["mean"])
        assert ok, f"mean scale {s}: max abs err {mx}, {nbad} outside tolerance"
    if check_bev:
        ok, mx, nbad = close(np_(vox["bev"]), ref["bev"])
        assert ok, f"bev: max abs err {mx}, {nbad} outside tolerance"
        assert np.array_equal(np_(vox["bev"]) != 0, ref["bev"] != 0)
    assert np.array_equal(np_(pg["vis_mask"]), ref["vis_mask"]), "vis_mask"
    assert np.array_equal(np_(pg["cam"]), ref["cam"]), "cam"
    ok, mx, nbad = close(np_(pg["uvd"]), ref["uvd"])
    assert ok, f"uvd: max abs err {mx}, {nbad} outside tolerance"
    ok, mx, nbad = close(np_(pg["gathered"]), ref["gathered"])
    assert ok, f"gathered: max abs err {mx}, {nbad} outside tolerance"
    assert np.array_equal(np_(rd["expert"]), ref["expert"]), "expert"
    assert np.array_equal(np_(rd["offsets"]), ref["offsets"]), "offsets"
    assert np.array_equal(np_(rd["perm"]), ref["perm"]), "perm"
    # rows are copies: compare bit patterns (inputs may hold NaN)
    assert np.array_equal(np_(rd["points_out"]).view(np.uint32), ref["points_out"].view(np.uint32)), "points_out"
    ok, mx, nbad = close(np_(rd["feat_out"]), ref["feat_out"])
    assert ok, f"feat_out: max abs err {mx}, {nbad} outside tolerance"
