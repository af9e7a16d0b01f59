"""CUDA library vs CPU oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import emc2_gen as gen
from parity import close, compare_bridge, np_, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b200():
    import paper_2507_04123_b200 as pkg
    from paper_2507_04123_b200 import build
    build.build()
    assert torch.cuda.is_available()
    return pkg


def run_case(pkg, oracle, w, batch=None, repeat=1, staged=False, tune=()):
    batch = batch if batch is not None else gen.make_batch(w)
    ref = oracle.bridge(w, batch)
    br = pkg.Bridge(pkg.config_from_workload(w))
    for knob, value in tune:
        br.set_tuning(knob, value)
    d = to_dev(batch)
    bufs = None
    step = br.run_staged if staged else br.run   # three calls, or emc2_bridge_run
    for _ in range(repeat):                      # a second call must see clean scratch
        bufs = step(d["points"], d["proj"], d["feat"], bufs)
    br.status()
    compare_bridge(w, ref, bufs)
    br.close()
    return ref, bufs


@pytest.mark.parametrize("staged", [False, True], ids=["one_call", "three_calls"])
@pytest.mark.parametrize("cid", [0, 1, 2, 3])
def test_benchmark_configs_match_the_oracle(b200, oracle, cid, staged):
    run_case(b200, oracle, gen.workload(cid), repeat=2, staged=staged)


@pytest.mark.parametrize("B,N", [(1, 1), (1, 255), (2, 257), (3, 1000), (2, 4099), (5, 777)])
def test_ragged_shapes(b200, oracle, B, N):
    for base in (gen.KITTI, gen.NUSCENES):
        run_case(b200, oracle, base.with_shape(B, N), repeat=2, staged=(N % 2 == 0))


TUNINGS = [(("row_store", 0),), (("row_store", 1),), (("row_store", 2),), (("row_store", 3),), (("mark_in_projection", 0),),
           (("mark_in_projection", 1),), (("split_batch", 0),), (("split_batch", 1),), (("dedup_fine", 1),), (("dedup_fine", 2),), (("dedup_pillars", 1),),
           (("dedup_pillars", 2),), (("dedup_fine", 2), ("dedup_pillars", 1)), (("dedup_fine", 1), ("dedup_pillars", 2))]


@pytest.mark.parametrize("tune", TUNINGS, ids=lambda t: "-".join(f"{k}{v}" for k, v in t))
def test_every_implementation_choice_matches_the_oracle(b200, oracle, tune):
    """The alternatives behind emc2_bridge_set_tuning produce the same outputs: full tiles, ragged tiles,
    both feature widths, the dense frame (cap binds), and a frame with an expert that owns nothing."""
    for w in (gen.NUSCENES.with_shape(2, 20000), gen.KITTI.with_shape(3, 4099), gen.NUSCENES.with_shape(1, 31),
              gen.DENSE.with_shape(1, 50000), gen.KITTI.with_shape(1, 1)):
        run_case(b200, oracle, w, repeat=2, tune=tune)
        run_case(b200, oracle, w, repeat=1, staged=True, tune=tune)
    w = gen.KITTI.with_shape(1, 3000)
    batch = gen.make_batch(w)
    batch["points"][..., 0] = np.abs(batch["points"][..., 0]) % 15.0     # everything nearer than 20 m
    batch["points"][..., 1] = batch["points"][..., 1] % 10.0
    run_case(b200, oracle, w, batch=batch, repeat=2, tune=tune)


def test_per_voxel_cap_on_the_fine_scale(b200, oracle):
    """max_points on a grid too large for per-cell counts (the fine scale): keep-first-by-index, counts = kept,
    means over the kept points, dropped points at -1 - as on the pillar scale."""
    from dataclasses import replace
    for base, n in ((gen.DENSE, 150_000), (gen.NUSCENES.with_shape(2, 80_000), None)):
        w = base if n is None else base.with_shape(1, n)
        w = replace(w, grids=(replace(w.grids[0], max_points=3), w.grids[1]))
        ref, bufs = run_case(b200, oracle, w, repeat=2)
        assert int((ref["vox0"]["counts"] == 3).sum()) > 100          # the cap binds on many voxels
        assert int((ref["vox0"]["point_voxel"] < 0).sum()) > 0
        run_case(b200, oracle, w, repeat=2, staged=True)


def test_one_call_without_the_side_stream(b200, oracle):
    w = gen.NUSCENES.with_shape(2, 20000)
    batch = gen.make_batch(w)
    ref = oracle.bridge(w, batch)
    br = b200.Bridge(b200.config_from_workload(w))
    br.set_overlap(False)                        # every kernel on the caller's stream
    d = to_dev(batch)
    bufs = br.run(d["points"], d["proj"], d["feat"])
    bufs = br.run(d["points"], d["proj"], d["feat"], bufs)
    br.status()
    compare_bridge(w, ref, bufs)
    br.set_overlap(True)
    bufs = br.run(d["points"], d["proj"], d["feat"], bufs)
    br.status()
    compare_bridge(w, ref, bufs)
    br.close()


def test_one_call_on_a_side_stream_of_the_caller(b200, oracle):
    # The call must order itself after work already queued on the caller's stream and be complete,
    # stage 1 included, for work queued after it on that stream.
    w = gen.KITTI.with_shape(2, 30000)
    batch = gen.make_batch(w)
    ref = oracle.bridge(w, batch)
    br = b200.Bridge(b200.config_from_workload(w))
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        d = {k: torch.from_numpy(v).pin_memory().to("cuda", non_blocking=True) for k, v in batch.items()}
        bufs = br.run(d["points"], d["proj"], d["feat"])
        host = {"nv": bufs["vox"]["num_voxels"].to("cpu", non_blocking=True),
                "bev": bufs["vox"]["bev"].to("cpu", non_blocking=True)}
    s.synchronize()
    assert host["nv"].tolist() == [ref["vox0"]["num_voxels"], ref["vox1"]["num_voxels"]]
    assert np.array_equal(host["bev"].numpy() != 0, ref["bev"] != 0)
    with torch.cuda.stream(s):
        br.status()
    compare_bridge(w, ref, bufs)
    br.close()


def test_one_call_without_the_rows_in_point_order(b200, oracle):
    w = gen.NUSCENES.with_shape(2, 30001)
    batch = gen.make_batch(w)
    ref = oracle.bridge(w, batch)
    br = b200.Bridge(b200.config_from_workload(w))
    d = to_dev(batch)
    bufs = br.run(d["points"], d["proj"], d["feat"])
    kept = bufs["pg"]["gathered"]
    kept.fill_(7.0)
    bufs["rd"]["feat_out"].fill_(-1.0)
    bufs["pg"]["gathered"] = None
    br.run(d["points"], d["proj"], d["feat"], bufs)
    br.status()
    assert bool((kept == 7.0).all())                 # not written
    bufs["pg"]["gathered"] = torch.from_numpy(ref["gathered"]).cuda()   # everything else as always
    compare_bridge(w, ref, bufs)
    br.close()


def test_one_call_from_host_buffers(b200, oracle):
    # pinned and pageable host memory; results come back into host tensors without a sync by the library
    w = gen.NUSCENES.with_shape(2, 20000)
    batch = gen.make_batch(w)
    ref = oracle.bridge(w, batch)
    br = b200.Bridge(b200.config_from_workload(w))
    d = to_dev(batch)
    bufs = br.run(d["points"], d["proj"], d["feat"])          # output buffers of the right shapes
    for pinned in (True, False):
        host = {k: torch.from_numpy(v.copy()) for k, v in batch.items()}
        if pinned:
            host = {k: v.pin_memory() for k, v in host.items()}
        staging = {k: torch.full_like(v, float("nan")) for k, v in d.items()}
        h_off = torch.full((w.B, w.num_experts + 1), -1, dtype=torch.int32)
        h_nv = torch.full((2,), -1, dtype=torch.int32)
        if pinned:
            h_off, h_nv = h_off.pin_memory(), h_nv.pin_memory()
        bufs["rd"]["feat_out"].fill_(-1.0)
        br.run_host(host, staging, bufs, h_off, h_nv)
        torch.cuda.synchronize()
        br.status()
        compare_bridge(w, ref, bufs)
        assert np.array_equal(h_off.numpy(), ref["offsets"])
        assert h_nv.tolist() == [ref["vox0"]["num_voxels"], ref["vox1"]["num_voxels"]]
        assert torch.equal(staging["points"].cpu(), host["points"])
    br.close()


def test_one_call_replays_from_a_cuda_graph(b200, oracle):
    # emc2_bridge_run only enqueues (kernels, a fork and a join by events), so a caller can capture
    # it once and replay it on new frames written into the same buffers.
    w = gen.KITTI.with_shape(2, 30000)
    first, second = gen.make_batch(w, frames=[0, 1]), gen.make_batch(w, frames=[2, 3])
    br = b200.Bridge(b200.config_from_workload(w))
    d = to_dev(first)
    bufs = br.run(d["points"], d["proj"], d["feat"])      # allocates the outputs, outside the capture
    br.status()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        br.run(d["points"], d["proj"], d["feat"], bufs)
    for batch in (second, first):
        for k, v in batch.items():
            d[k].copy_(torch.from_numpy(v))
        bufs["pg"]["gathered"].fill_(-1.0)
        bufs["vox"]["num_voxels"].fill_(-1)
        graph.replay()
        torch.cuda.synchronize()
        br.status()
        compare_bridge(w, oracle.bridge(w, batch), bufs)
    del graph
    # the stage calls and the optional calls, one after another in a second graph
    vi = br.voxel_image(bufs["vox"], 0, bufs["pg"]["vis_mask"], bufs["pg"]["gathered"])
    rb = br.rulebook(bufs["vox"], 0)
    oc = br.occlusion(d["points"], d["proj"], bufs["pg"]["vis_mask"], 8, 0.5)
    pooled = br.pool_features(d["feat"], 2)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        br.run_staged(d["points"], d["proj"], d["feat"], bufs)
        br.voxel_image(bufs["vox"], 0, bufs["pg"]["vis_mask"], bufs["pg"]["gathered"], vi)
        br.rulebook(bufs["vox"], 0, out=rb)
        br.occlusion(d["points"], d["proj"], bufs["pg"]["vis_mask"], 8, 0.5, oc)
        br.pool_features(d["feat"], 2, out=pooled)
    for k, v in second.items():
        d[k].copy_(torch.from_numpy(v))
    for t in (rb["rule_in"], oc["occ_mask"], vi["vox_img_count"]):
        t.fill_(-1 if t.dtype != torch.uint8 else 255)
    graph.replay()
    torch.cuda.synchronize()
    br.status()
    ref = oracle.bridge(w, second)
    compare_bridge(w, ref, bufs)
    M = ref["vox0"]["num_voxels"]
    off, rin, rout = oracle.rulebook(ref["vox0"]["coords"][:M])
    assert np.array_equal(np_(rb["offsets"]), off) and np.array_equal(np_(rb["rule_in"])[:off[27]], rin)
    _, cnt = oracle.voxel_image(ref["vox0"]["point_voxel"], M, ref["vis_mask"], ref["gathered"])
    assert np.array_equal(np_(vi["vox_img_count"])[:M], cnt)
    _, want_occ, _ = oracle.occlusion(second["points"], second["proj"], w.img_h, w.img_w, ref["vis_mask"], 8, 0.5)
    assert np.array_equal(np_(oc["occ_mask"]), want_occ)
    assert np.abs(np_(pooled).astype(np.float64) - oracle.pool(second["feat"], 2)).max() <= 1e-5
    del graph
    br.close()


def test_planar_maps_to_channels_last(b200, oracle):
    rng = np.random.default_rng(21)
    from dataclasses import replace
    # pixel counts with and without 16-byte aligned channel rows; channel counts that fill a
    # 64-channel tile, leave a 16- and a 4-channel remainder, or are one half group
    for base in (gen.KITTI.with_shape(2, 100), gen.NUSCENES.with_shape(1, 100), gen.TINY,
                 replace(gen.NUSCENES.with_shape(1, 100), feat_c=68), replace(gen.TINY, feat_c=12),
                 replace(gen.TINY, feat_c=4, img_w=1250)):
        br = b200.Bridge(b200.config_from_workload(base))
        planar = rng.standard_normal((base.B, base.K, base.feat_c, base.feat_h, base.feat_w)).astype(np.float32)
        got = br.features_channels_last(torch.from_numpy(planar).cuda())
        br.status()
        assert np.array_equal(np_(got), oracle.channels_last(planar))
        br.close()


@pytest.mark.parametrize("p", [1, 2, 4])
def test_multiscale_pooling_and_the_pooled_path(b200, oracle, p):
    from dataclasses import replace
    for base in (gen.KITTI.with_shape(2, 6000), gen.NUSCENES.with_shape(1, 9000)):
        batch = gen.make_batch(base)
        d = to_dev(batch)
        br = b200.Bridge(b200.config_from_workload(base))
        pooled = br.pool_features(d["feat"], p)
        br.status()
        want = oracle.pool(batch["feat"], p)
        assert tuple(pooled.shape) == want.shape
        assert np.abs(np_(pooled).astype(np.float64) - want).max() <= 1e-5
        br.close()
        # the whole bridge on the pooled maps: texels at the window centres, stride p * s
        w = replace(base, feat_stride=base.feat_stride * p, feat_offset=(p - 1) / 2 * base.feat_stride)
        assert (w.feat_h, w.feat_w) == want.shape[2:4]
        pbatch = dict(batch, feat=want)
        ref = oracle.bridge(w, pbatch)
        br = b200.Bridge(b200.config_from_workload(w))
        dp = to_dev(pbatch)
        for step in (br.run, br.run_staged):
            bufs = step(dp["points"], dp["proj"], dp["feat"])
            br.status()
            compare_bridge(w, ref, bufs)
        br.close()


@pytest.mark.parametrize("cid,B,N", [(2, 2, 50_000), (1, 3, 33_333), (3, 1, 300_000), (2, 1, 1)])
def test_image_features_per_voxel(b200, oracle, cid, B, N):
    w = gen.workload(cid).with_shape(B, N)
    batch = gen.make_batch(w)
    ref = oracle.bridge(w, batch)
    br = b200.Bridge(b200.config_from_workload(w))
    d = to_dev(batch)
    bufs = br.run(d["points"], d["proj"], d["feat"])
    for rep in range(2):                           # twice: the lists must not depend on old cursors
        for s in range(2):
            out = br.voxel_image(bufs["vox"], s, bufs["pg"]["vis_mask"], bufs["pg"]["gathered"])
            br.status()
            M = ref[f"vox{s}"]["num_voxels"]
            want, cnt = oracle.voxel_image(ref[f"vox{s}"]["point_voxel"], M, ref["vis_mask"], ref["gathered"])
            assert np.array_equal(np_(out["vox_img_count"])[:M], cnt), s
            ok, mx, nbad = close(np_(out["vox_img"])[:M], want)
            assert ok, f"scale {s}: max abs err {mx}, {nbad} outside tolerance"
            assert not np_(out["vox_img"])[:M][cnt == 0].any()
            # the same rows without the per-point buffer: blended from the maps voxel by voxel
            out = br.voxel_image_sampled(bufs["vox"], s, bufs["pg"]["uvd"], bufs["pg"]["cam"], d["feat"])
            br.status()
            assert np.array_equal(np_(out["vox_img_count"])[:M], cnt), s
            ok, mx, nbad = close(np_(out["vox_img"])[:M], want)
            assert ok, f"sampled, scale {s}: max abs err {mx}, {nbad} outside tolerance"
            assert not np_(out["vox_img"])[:M][cnt == 0].any()
    br.close()


@pytest.mark.parametrize("p", [2, 4])
def test_pooled_image_features_per_voxel(b200, oracle, p):
    """Multiscale Pooling and the fusion by voxel as ONE path, in the paper's order: pool the maps, sample them
    at the projected points, attach the rows to the voxels (zero rows where a voxel has no pixel).  The oracle
    chain is pool -> gather(window-centre offset) -> voxel_image; the CUDA chain is emc2_pool_features -> a
    handle for the pooled maps -> emc2_voxel_image_sampled, and emc2_voxel_image_pooled, which folds the
    pooling into the sampling and must agree with it."""
    from dataclasses import replace
    for base in (gen.NUSCENES.with_shape(2, 40_000), gen.KITTI.with_shape(1, 30_000)):
        batch = gen.make_batch(base)
        d = to_dev(batch)
        br0 = b200.Bridge(b200.config_from_workload(base))
        pooled = br0.pool_features(d["feat"], p)
        raw = br0.run(d["points"], d["proj"], d["feat"])         # unpooled handle: voxels, uvd, cam
        br0.status()
        w = replace(base, feat_stride=base.feat_stride * p, feat_offset=(p - 1) / 2 * base.feat_stride)
        ref = oracle.bridge(w, dict(batch, feat=oracle.pool(batch["feat"], p)))
        br = b200.Bridge(b200.config_from_workload(w))
        bufs = br.run(d["points"], d["proj"], pooled)
        br.status()
        for s in range(2):
            M = ref[f"vox{s}"]["num_voxels"]
            want, cnt = oracle.voxel_image(ref[f"vox{s}"]["point_voxel"], M, ref["vis_mask"], ref["gathered"])
            assert int((cnt == 0).sum()) > 0 and int((cnt > 1).sum()) > 0
            outs = {"pool, then sample per voxel": br.voxel_image_sampled(bufs["vox"], s, bufs["pg"]["uvd"],
                                                                          bufs["pg"]["cam"], pooled),
                    "pool, gather per point, then mean per voxel": br.voxel_image(bufs["vox"], s, bufs["pg"]["vis_mask"],
                                                                                  bufs["pg"]["gathered"]),
                    "pooling folded into the sampling": br0.voxel_image_pooled(raw["vox"], s, raw["pg"]["uvd"],
                                                                               raw["pg"]["cam"], d["feat"], p)}
            br.status()
            br0.status()
            for name, out in outs.items():
                assert np.array_equal(np_(out["vox_img_count"])[:M], cnt), (name, s)
                ok, mx, nbad = close(np_(out["vox_img"])[:M], want)
                assert ok, f"{name}, scale {s}, p {p}: max abs err {mx}, {nbad} outside tolerance"
                assert not np_(out["vox_img"])[:M][cnt == 0].any(), name
        br.close()
        br0.close()


def test_per_voxel_fusion_rejects_counts_of_another_batch(b200, oracle):
    # counts that add up to more than the points would make the per-voxel lists overrun their array:
    # the scan sees it, nothing is written and the status says so
    w = gen.KITTI.with_shape(1, 20_000)
    batch = gen.make_batch(w)
    br = b200.Bridge(b200.config_from_workload(w))
    d = to_dev(batch)
    bufs = br.run(d["points"], d["proj"], d["feat"])
    br.status()
    good = br.voxel_image(bufs["vox"], 0, bufs["pg"]["vis_mask"], bufs["pg"]["gathered"])
    br.status()
    wrong = {k: v for k, v in bufs["vox"].items()}
    wrong["counts"] = [torch.full_like(bufs["vox"]["counts"][0], 1 << 30), bufs["vox"]["counts"][1]]
    out = {"vox_img": torch.full_like(good["vox_img"], 3.0), "vox_img_count": torch.full_like(good["vox_img_count"], -5)}
    br.voxel_image(wrong, 0, bufs["pg"]["vis_mask"], bufs["pg"]["gathered"], out)
    assert br.status(raise_on_error=False) == b200.bridge.EMC2_ERR_INVALID_ARG
    assert bool((out["vox_img"] == 3.0).all()) and bool((out["vox_img_count"] == -5).all())
    br.voxel_image_sampled(wrong, 0, bufs["pg"]["uvd"], bufs["pg"]["cam"], d["feat"], out)
    assert br.status(raise_on_error=False) == b200.bridge.EMC2_ERR_INVALID_ARG
    assert bool((out["vox_img"] == 3.0).all())
    again = br.voxel_image(bufs["vox"], 0, bufs["pg"]["vis_mask"], bufs["pg"]["gathered"])   # and it recovers
    br.status()
    M = int(bufs["vox"]["num_voxels"][0].item())             # rows past the voxels found are not written
    assert torch.equal(again["vox_img_count"][:M], good["vox_img_count"][:M])
    br.close()


def test_per_voxel_fusion_with_counts_moved_between_voxels_reads_only_what_it_appended(b200, oracle):
    # counts with the right total but the wrong voxels (another scale's, or a stale buffer): a voxel must not
    # walk past the entries this call appended for it, so every row is a mean of rows of THIS batch
    w = gen.KITTI.with_shape(1, 20_000)
    batch = gen.make_batch(w)
    br = b200.Bridge(b200.config_from_workload(w))
    d = to_dev(batch)
    bufs = br.run(d["points"], d["proj"], d["feat"])
    br.status()
    pg = bufs["pg"]
    pg["gathered"].fill_(1.0)                                # every row of this batch is all ones
    M = int(bufs["vox"]["num_voxels"][0].item())
    wrong = {k: v for k, v in bufs["vox"].items()}
    moved = bufs["vox"]["counts"][0].clone()
    moved[:M] = torch.roll(moved[:M], 1)                     # same sum, other voxels
    wrong["counts"] = [moved, bufs["vox"]["counts"][1]]
    for call in (lambda: br.voxel_image(wrong, 0, pg["vis_mask"], pg["gathered"]),):
        out = call()
        assert br.status(raise_on_error=False) == b200.bridge.EMC2_OK
        rows = out["vox_img"][:M]
        cnt = out["vox_img_count"][:M]
        assert bool(torch.isfinite(rows).all())
        seen = cnt > 0
        assert bool((rows[seen] == 1.0).all()) and bool((rows[~seen] == 0.0).all())
    br.close()


@pytest.mark.parametrize("cid,B,N", [(2, 2, 60_000), (1, 3, 33_333), (3, 1, 150_000), (0, 1, 16_384), (2, 1, 1)])
def test_sparse_convolution_rulebook(b200, oracle, cid, B, N):
    w = gen.workload(cid).with_shape(B, N)
    batch = gen.make_batch(w)
    ref = oracle.bridge(w, batch)
    br = b200.Bridge(b200.config_from_workload(w))
    d = to_dev(batch)
    bufs = br.run(d["points"], d["proj"], d["feat"])
    for s in range(2):                             # the two scales use the two kinds of cell store
        M = ref[f"vox{s}"]["num_voxels"]
        off, rin, rout = oracle.rulebook(ref[f"vox{s}"]["coords"][:M])
        for rep in range(2):                       # twice: the store must be clean again after a call
            out = br.rulebook(bufs["vox"], s)
            br.status()
            assert np.array_equal(np_(out["offsets"]), off), s
            assert np.array_equal(np_(out["rule_in"])[:off[27]], rin), s
            assert np.array_equal(np_(out["rule_out"])[:off[27]], rout), s
    # and the voxelizer still finds its store all zero
    bufs = br.run(d["points"], d["proj"], d["feat"], bufs)
    br.status()
    compare_bridge(w, ref, bufs)
    br.close()


def test_rulebook_at_full_size(b200, oracle):
    """The benchmark's batch: properties that hold at any size, and the first frame pair by pair."""
    w = gen.NUSCENES
    batch = gen.make_batch(w, feature_frames=1)
    br = b200.Bridge(b200.config_from_workload(w))
    d = to_dev(batch)
    vox = br.voxelize(d["points"])
    out = br.rulebook(vox, 0)
    br.status()
    M = int(vox["num_voxels"][0].item())
    coords = np_(vox["coords"][0])[:M].astype(np.int64)
    off = np_(out["offsets"]).astype(np.int64)
    total = int(off[27])
    rin, rout = np_(out["rule_in"])[:total].astype(np.int64), np_(out["rule_out"])[:total].astype(np.int64)
    assert off[0] == 0 and np.all(np.diff(off) >= 0)
    assert rin.min() >= 0 and rin.max() < M and rout.min() >= 0 and rout.max() < M
    for k in range(27):
        i, o = rin[off[k]:off[k + 1]], rout[off[k]:off[k + 1]]
        shift = np.array([0, k // 9 - 1, (k // 3) % 3 - 1, k % 3 - 1])
        assert np.array_equal(coords[i], coords[o] + shift), k       # every listed pair is a true neighbour pair
        assert np.all(np.diff(o) > 0), k                              # ascending, no pair twice
        assert off[k + 1] - off[k] == off[27 - k] - off[26 - k], k    # as many as for the opposite offset
    assert np.array_equal(rin[off[13]:off[14]], np.arange(M))
    # frames never pair with one another, so the first frame's rows form the rulebook of its own list
    M0 = int((coords[:, 0] == 0).sum())
    want_off, want_in, want_out = oracle.rulebook(coords[:M0].astype(np.int32))
    for k in range(27):
        i, o = rin[off[k]:off[k + 1]], rout[off[k]:off[k + 1]]
        n = int(np.searchsorted(o, M0))
        assert n == want_off[k + 1] - want_off[k], k
        assert np.array_equal(i[:n], want_in[want_off[k]:want_off[k + 1]]), k
        assert np.array_equal(o[:n], want_out[want_off[k]:want_off[k + 1]]), k
    br.close()


def test_rulebook_errors_only_the_device_sees(b200, oracle):
    w = gen.KITTI.with_shape(1, 20_000)
    batch = gen.make_batch(w)
    ref = oracle.bridge(w, batch)
    br = b200.Bridge(b200.config_from_workload(w))
    d = to_dev(batch)
    bufs = br.run(d["points"], d["proj"], d["feat"])
    br.status()
    M = ref["vox0"]["num_voxels"]
    off, rin, rout = oracle.rulebook(ref["vox0"]["coords"][:M])
    total = int(off[27])
    # too few pair slots: the true count is reported, nothing is written past the end
    small = total // 2
    guard = 64
    out = {"offsets": torch.empty(28, dtype=torch.int32, device="cuda"),
           "rule_in": torch.full((small + guard,), -7, dtype=torch.int32, device="cuda"),
           "rule_out": torch.full((small + guard,), -7, dtype=torch.int32, device="cuda")}
    view = {"offsets": out["offsets"], "rule_in": out["rule_in"][:small], "rule_out": out["rule_out"][:small]}
    br.rulebook(bufs["vox"], 0, out=view)
    assert br.status(raise_on_error=False) == b200.bridge.EMC2_ERR_CAPACITY
    assert np.array_equal(np_(out["offsets"]), off)
    assert (np_(out["rule_in"])[small:] == -7).all() and (np_(out["rule_out"])[small:] == -7).all()
    # every pair slot below the end that belongs to a written position holds the right pair
    got_in, got_out = np_(out["rule_in"])[:small], np_(out["rule_out"])[:small]
    assert np.array_equal(got_in, rin[:small]) and np.array_equal(got_out, rout[:small])
    # a list that is not in ascending order is reported, and the store is clean afterwards
    bad = {"coords": [bufs["vox"]["coords"][0].clone(), bufs["vox"]["coords"][1]], "num_voxels": bufs["vox"]["num_voxels"]}
    bad["coords"][0][[5, 9]] = bad["coords"][0][[9, 5]]
    br.rulebook(bad, 0)
    assert br.status(raise_on_error=False) == b200.bridge.EMC2_ERR_INVALID_ARG
    out = br.rulebook(bufs["vox"], 0)
    br.status()
    assert np.array_equal(np_(out["rule_in"])[:total], rin) and np.array_equal(np_(out["rule_out"])[:total], rout)
    br.close()


@pytest.mark.parametrize("cid,B,N,cell,margin", [(2, 2, 120_000, 8, 0.5), (1, 3, 40_001, 4, 0.25),
                                                 (3, 1, 300_000, 16, 1.0), (2, 1, 5000, 64, 0.0)])
def test_occlusion_and_routing_of_occluded_points(b200, oracle, cid, B, N, cell, margin):
    w = gen.workload(cid).with_shape(B, N)
    batch = gen.make_batch(w)
    ref = oracle.bridge(w, batch)
    zbuf, occ, clear = oracle.occlusion(batch["points"], batch["proj"], w.img_h, w.img_w, ref["vis_mask"], cell, margin)
    br = b200.Bridge(b200.config_from_workload(w))
    d = to_dev(batch)
    bufs = br.run(d["points"], d["proj"], d["feat"])
    out = None
    for _ in range(2):
        out = br.occlusion(d["points"], d["proj"], bufs["pg"]["vis_mask"], cell, margin, out)
    br.status()
    assert np.array_equal(np_(out["zbuf"]).view(np.uint32), zbuf.view(np.uint32))      # exact, +inf included
    assert np.array_equal(np_(out["occ_mask"]), occ)
    assert np.array_equal(np_(out["clear_mask"]), clear)
    assert occ.any()
    # occluded points routed as not visible
    rd = br.route_dispatch(d["points"], out["clear_mask"], bufs["pg"]["gathered"])
    br.status()
    ex = oracle.route(batch["points"], clear, w.thresholds, w.lut)
    off, perm, _, _ = oracle.dispatch(ex, batch["points"], ref["gathered"], w.num_experts)
    assert np.array_equal(np_(rd["expert"]), ex) and np.array_equal(np_(rd["offsets"]), off)
    assert np.array_equal(np_(rd["perm"]), perm)
    assert (ex != ref["expert"]).any()
    br.close()


def test_scene_route_matches_the_oracle(b200, oracle):
    w = gen.NUSCENES.with_shape(5, 4000)
    batch = gen.make_batch(w)
    p = batch["points"]
    p[1, :, :2] *= 0.2                           # everything near: no far expert in this frame
    p[2, :, 0] = -400.0                          # everything beyond 50 m and invisible
    p[3, 1:, :2] *= 0.1
    p[3, 0, :3] = (60.0, 0.0, 0.0)               # a single far point
    ref = oracle.bridge(w, batch)
    br = b200.Bridge(b200.config_from_workload(w))
    d = to_dev(batch)
    bufs = br.run(d["points"], d["proj"], d["feat"])
    for pr, mp in (((0, 1, 2, 3), 1), ((0, 1, 2, 3), 2), ((3, 2, 1, 0), 1), ((1, 1, 1, 1), 1), ((0, 2, 1, 2), 50)):
        got = np_(br.scene_route(bufs["rd"]["offsets"], pr, mp))
        assert np.array_equal(got, oracle.scene_route(ref["offsets"], pr, mp)), (pr, mp)
    assert len(set(oracle.scene_route(ref["offsets"], (0, 1, 2, 3), 1).tolist())) > 1
    empty = torch.zeros((5, w.num_experts + 1), dtype=torch.int32, device="cuda")
    assert (np_(br.scene_route(empty, (0, 1, 2, 3))) == -1).all()
    br.status()
    br.close()


def test_sweep_cell_with_six_cameras(b200, oracle):
    run_case(b200, oracle, gen.SWEEP.with_shape(2, 65536))


def test_largest_sweep_cell_on_sampled_frames(b200, oracle):
    """32 frames x 524,288 points (the largest size a handle accepts), checked on two of the frames.

    Frames are independent, so the oracle is run on the sampled frames alone and every output of
    those frames is compared: voxel rows through their frame column, the rest by slicing."""
    w = gen.SWEEP.with_shape(32, 524288)
    sample = [5, 31]
    pts = np.empty((w.B, w.N, w.C), np.float32)
    for f in range(w.B):
        pts[f] = gen.make_points(w, f % 4)               # four distinct clouds, repeated
    pts[sample[1]] = gen.make_points(w, 7)               # and one frame of its own
    proj = np.broadcast_to(gen.make_projection(w), (w.B, w.K, 3, 4)).copy()
    fmap = gen.make_features(w, 0)
    dev = "cuda"
    d_pts, d_proj = torch.from_numpy(pts).to(dev), torch.from_numpy(proj).to(dev)
    d_feat = torch.from_numpy(fmap).to(dev)[None].expand(w.B, -1, -1, -1, -1).contiguous()
    br = b200.Bridge(b200.config_from_workload(w))
    bufs = br.run(d_pts, d_proj, d_feat)
    br.status()
    sub = w.with_shape(len(sample), w.N)
    ref = oracle.bridge(sub, {"points": pts[sample], "proj": proj[sample],
                              "feat": np.broadcast_to(fmap, (len(sample),) + fmap.shape).copy()})
    vox = bufs["vox"]
    nv = np_(vox["num_voxels"])
    for s in range(2):
        coords = np_(vox["coords"][s])[:nv[s]]
        counts = np_(vox["counts"][s])[:nv[s]]
        mean = np_(vox["mean"][s])[:nv[s]]
        pv = np_(vox["point_voxel"][s])
        r = ref[f"vox{s}"]
        for k, f in enumerate(sample):
            rows = np.nonzero(coords[:, 0] == f)[0]
            want = r["coords"][:, 0] == k
            assert len(rows) == want.sum()
            assert np.array_equal(coords[rows, 1:], r["coords"][want, 1:])
            assert np.array_equal(counts[rows], r["counts"][want])
            assert close(mean[rows], r["mean"][want])[0]
            first = rows[0] if len(rows) else 0
            base = np.nonzero(want)[0][0] if len(rows) else 0
            got_pv, want_pv = pv[f], r["point_voxel"][k]
            assert np.array_equal(got_pv >= 0, want_pv >= 0)
            assert np.array_equal(got_pv[got_pv >= 0] - first, want_pv[want_pv >= 0] - base)
    assert close(np_(vox["bev"][sample]), ref["bev"])[0]
    pg, rd = bufs["pg"], bufs["rd"]
    for name in ("vis_mask", "cam"):
        assert np.array_equal(np_(pg[name][sample]), ref[name]), name
    for name in ("expert", "offsets", "perm"):
        assert np.array_equal(np_(rd[name][sample]), ref[name]), name
    assert close(np_(pg["uvd"][sample]), ref["uvd"])[0]
    assert close(np_(pg["gathered"][sample]), ref["gathered"])[0]
    assert close(np_(rd["feat_out"][sample]), ref["feat_out"])[0]
    assert np.array_equal(np_(rd["points_out"][sample]).view(np.uint32), ref["points_out"].view(np.uint32))
    br.close()


def test_degenerate_frames(b200, oracle):
    w = gen.NUSCENES.with_shape(2, 3000)
    batch = gen.make_batch(w)
    p = batch["points"]
    p[0, :, :3] = (1.0, 2.0, 0.5)                # every point of frame 0 in one voxel (cap binds)
    p[1, :1000, 0] = 500.0                       # outside both grids, beyond every threshold
    p[1, 1000:1100, 1] = np.nan                  # non-finite coordinates
    p[1, 1100:1200, 2] = np.inf
    run_case(b200, oracle, w, batch)
    q = gen.make_batch(w)
    q["points"][..., :3] = 1e6                   # nothing in range, nothing visible: zero voxels
    ref, bufs = run_case(b200, oracle, w, q)
    assert ref["vox0"]["num_voxels"] == 0 and ref["vox1"]["num_voxels"] == 0
    assert not np_(bufs["vox"]["bev"]).any()


def test_single_expert_and_empty_expert(b200, oracle):
    from dataclasses import replace
    w = replace(gen.KITTI.with_shape(2, 5000), lut=((2, 2, 2, 0, 0, 0, 0, 0), (2, 2, 2, 0, 0, 0, 0, 0)))
    ref, _ = run_case(b200, oracle, w)
    assert (ref["offsets"][:, 2] == 0).all() and (ref["offsets"][:, 3] == w.N).all()


@pytest.mark.parametrize("design", [0, 1, 2], ids=["direct", "hash", "sort"])
def test_empty_inputs(b200, design):
    w = gen.KITTI.with_shape(2, 64)
    br = b200.Bridge(b200.config_from_workload(w))
    br.set_tuning("dedup_fine", design)
    br.set_tuning("dedup_pillars", design)
    for B, N in ((0, 64), (2, 0)):
        pts = torch.zeros((B, N, 4), device="cuda")
        proj = torch.zeros((B, 1, 3, 4), device="cuda")
        feat = torch.zeros((B, 1, w.feat_h, w.feat_w, w.feat_c), device="cuda")
        bufs = br.run(pts, proj, feat)
        br.status()
        assert np_(bufs["vox"]["num_voxels"]).tolist() == [0, 0]
        if B:
            assert (np_(bufs["rd"]["offsets"]) == 0).all()
            assert not np_(bufs["vox"]["bev"]).any()       # an image without points is all zero
    br.close()


def test_capacity_overflow_is_reported_and_handle_recovers(b200, oracle):
    w = gen.TINY
    batch = gen.make_batch(w)
    ref = oracle.bridge(w, batch)
    br = b200.Bridge(b200.config_from_workload(w))
    d = to_dev(batch)
    cap = [1000, 500]
    out = br.voxelize(d["points"], capacity=cap)
    assert br.status(raise_on_error=False) == b200.bridge.EMC2_ERR_CAPACITY
    nv = np_(out["num_voxels"])
    assert nv[0] == ref["vox0"]["num_voxels"] and nv[1] == ref["vox1"]["num_voxels"]   # true counts
    for s in range(2):
        assert np.array_equal(np_(out["coords"][s])[:cap[s]], ref[f"vox{s}"]["coords"][:cap[s]])
        assert np.array_equal(np_(out["counts"][s])[:cap[s]], ref[f"vox{s}"]["counts"][:cap[s]])
    assert br.status(raise_on_error=False) == 0                   # sticky word was cleared
    bufs = br.run(d["points"], d["proj"], d["feat"])              # scratch is clean again
    br.status()
    compare_bridge(w, ref, bufs)
    br.close()


def test_integer_outputs_are_deterministic(b200):
    w = gen.DENSE
    d = to_dev(gen.make_batch(w))
    br = b200.Bridge(b200.config_from_workload(w))
    runs = []
    for _ in range(2):
        bufs = br.run(d["points"], d["proj"], d["feat"])
        br.status()
        nv = np_(bufs["vox"]["num_voxels"])
        runs.append([np_(bufs["vox"]["coords"][1])[:nv[1]].copy(), np_(bufs["vox"]["counts"][1])[:nv[1]].copy(),
                     np_(bufs["vox"]["point_voxel"][1]).copy(), np_(bufs["rd"]["perm"]).copy(),
                     np_(bufs["pg"]["vis_mask"]).copy()])
    for a, b in zip(*runs):
        assert np.array_equal(a, b)
    br.close()


def test_host_detected_errors(b200):
    w = gen.TINY
    br = b200.Bridge(b200.config_from_workload(w))
    pts = torch.zeros((1, w.N + 1, 4), device="cuda")
    with pytest.raises(b200.Emc2Error) as e:
        br.voxelize(pts)
    assert e.value.status == b200.bridge.EMC2_ERR_INVALID_ARG
    pts = torch.zeros((1, 65, 4), device="cuda").view(-1)[1:257].view(1, 64, 4)   # misaligned view
    with pytest.raises((b200.Emc2Error, ValueError)):
        br.voxelize(pts)
    br.close()
