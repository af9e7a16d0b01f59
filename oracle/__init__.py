"""ctypes front end of the CPU oracle (test infrastructure only).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  The CUDA library and its Python binding never do.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, Optional, Sequence

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "emc2_oracle.cpp")
_LIB = os.path.join(_DIR, "libemc2_oracle.so")
_lib: Optional[ctypes.CDLL] = None

_F = ctypes.POINTER(ctypes.c_float)
_I = ctypes.POINTER(ctypes.c_int32)
_U8 = ctypes.POINTER(ctypes.c_uint8)
_I8 = ctypes.POINTER(ctypes.c_int8)


def build(force: bool = False) -> str:
    """Compile the oracle with contraction off and no fast-math."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
               "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.emc2o_voxelize.restype = ctypes.c_int
        _lib.emc2o_rulebook.restype = ctypes.c_longlong
    return _lib


def _p(a: np.ndarray, t):
    return a.ctypes.data_as(t)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def voxelize(points: np.ndarray, grid_min: Sequence[float], voxel: Sequence[float],
             dims: Sequence[int], cap: int = 0) -> Dict[str, np.ndarray]:
    """One grid scale: unique voxels in canonical order, counts, means, inverse map."""
    points = _f32(points)
    B, N, C = points.shape
    mn, vs = _f32(grid_min), _f32(voxel)
    dm = np.ascontiguousarray(dims, dtype=np.int32)
    tot = B * N
    coords = np.empty((tot, 4), np.int32)
    counts = np.empty(tot, np.int32)
    mean = np.empty((tot, C), np.float32)
    pv = np.empty((B, N), np.int32)
    M = lib().emc2o_voxelize(B, N, C, _p(points, _F), _p(mn, _F), _p(vs, _F), _p(dm, _I), int(cap),
                             _p(coords, _I), _p(counts, _I), _p(mean, _F), _p(pv, _I))
    return {"num_voxels": M, "coords": coords[:M].copy(), "counts": counts[:M].copy(),
            "mean": mean[:M].copy(), "point_voxel": pv}


def bev(B: int, C: int, Gy: int, Gx: int, coords: np.ndarray, mean: np.ndarray) -> np.ndarray:
    coords = np.ascontiguousarray(coords, np.int32)
    mean = _f32(mean)
    out = np.empty((B, C, Gy, Gx), np.float32)
    lib().emc2o_bev(B, C, Gy, Gx, len(coords), _p(coords, _I), _p(mean, _F), _p(out, _F))
    return out


def project(points: np.ndarray, proj: np.ndarray, H: int, W: int, min_depth: float):
    points, proj = _f32(points), _f32(proj)
    B, N, C = points.shape
    K = proj.shape[1]
    uvd = np.empty((B, N, 3), np.float32)
    mask = np.empty((B, N), np.uint8)
    cam = np.empty((B, N), np.int8)
    lib().emc2o_project(B, N, C, K, _p(points, _F), _p(proj, _F), H, W, ctypes.c_float(min_depth),
                        _p(uvd, _F), _p(mask, _U8), _p(cam, _I8))
    return uvd, mask, cam


def channels_last(planar: np.ndarray) -> np.ndarray:
    """[B,K,Cf,Hf,Wf] -> [B,K,Hf,Wf,Cf] (a copy)."""
    planar = _f32(planar)
    B, K, Cf, Hf, Wf = planar.shape
    out = np.empty((B, K, Hf, Wf, Cf), np.float32)
    lib().emc2o_channels_last(B * K, Cf, Hf, Wf, _p(planar, _F), _p(out, _F))
    return out


def pool(feat: np.ndarray, p: int) -> np.ndarray:
    """p x p average pooling of channels-last feature maps (Sec. 3.5, Multiscale Pooling)."""
    feat = _f32(feat)
    B, K, Hf, Wf, Cf = feat.shape
    out = np.empty((B, K, -(-Hf // p), -(-Wf // p), Cf), np.float32)
    lib().emc2o_pool(B, K, Hf, Wf, Cf, int(p), _p(feat, _F), _p(out, _F))
    return out


def gather(uvd: np.ndarray, cam: np.ndarray, feat: np.ndarray, stride: int, offset: float = 0.0) -> np.ndarray:
    uvd, feat = _f32(uvd), _f32(feat)
    cam = np.ascontiguousarray(cam, np.int8)
    B, N, _ = uvd.shape
    _, K, Hf, Wf, Cf = feat.shape
    out = np.empty((B, N, Cf), np.float32)
    lib().emc2o_gather(B, N, K, Hf, Wf, Cf, int(stride), ctypes.c_float(offset), _p(uvd, _F), _p(cam, _I8),
                       _p(feat, _F), _p(out, _F))
    return out


def route(points: np.ndarray, vis_mask: np.ndarray, thresholds: Sequence[float],
          lut: Sequence[Sequence[int]]) -> np.ndarray:
    points = _f32(points)
    B, N, C = points.shape
    vis_mask = np.ascontiguousarray(vis_mask, np.uint8)
    th = _f32(thresholds)
    l = np.zeros((2, 8), np.uint8)
    for v in range(2):
        row = list(lut[v])[:8]
        l[v, :len(row)] = row
    out = np.empty((B, N), np.uint8)
    lib().emc2o_route(B, N, C, _p(points, _F), _p(vis_mask, _U8), len(th), _p(th, _F), _p(l, _U8),
                      _p(out, _U8))
    return out


def dispatch(expert: np.ndarray, points: np.ndarray, gathered: np.ndarray, num_experts: int):
    points, gathered = _f32(points), _f32(gathered)
    expert = np.ascontiguousarray(expert, np.uint8)
    B, N, C = points.shape
    Cf = gathered.shape[2]
    E = int(num_experts)
    assert int(expert.max(initial=0)) < E
    offsets = np.empty((B, E + 1), np.int32)
    perm = np.empty((B, N), np.int32)
    pout = np.empty_like(points)
    fout = np.empty_like(gathered)
    lib().emc2o_dispatch(B, N, C, Cf, E, _p(expert, _U8), _p(points, _F), _p(gathered, _F),
                         _p(offsets, _I), _p(perm, _I), _p(pout, _F), _p(fout, _F))
    return offsets, perm, pout, fout


def voxel_image(point_voxel: np.ndarray, num_voxels: int, vis_mask: np.ndarray, gathered: np.ndarray):
    """Image features per voxel (Fig. 5): mean gathered row of the voxel's visible points, else zeros."""
    pv = np.ascontiguousarray(point_voxel, np.int32).reshape(-1)
    vis = np.ascontiguousarray(vis_mask, np.uint8).reshape(-1)
    g = _f32(gathered).reshape(len(pv), -1)
    M, Cf = int(num_voxels), g.shape[1]
    out = np.empty((M, Cf), np.float32)
    cnt = np.empty(M, np.int32)
    lib().emc2o_voxel_image(ctypes.c_longlong(len(pv)), M, Cf, _p(pv, _I), _p(vis, _U8), _p(g, _F), _p(out, _F),
                            _p(cnt, _I))
    return out, cnt


def occlusion(points: np.ndarray, proj: np.ndarray, H: int, W: int, vis_mask: np.ndarray, cell: int,
              margin: float):
    """Depth-buffer occlusion per camera: (zbuf [B,K,Hz,Wz], occ_mask, clear_mask)."""
    points, proj = _f32(points), _f32(proj)
    B, N, C = points.shape
    K = proj.shape[1]
    vis = np.ascontiguousarray(vis_mask, np.uint8)
    Hz, Wz = -(-H // cell), -(-W // cell)
    zbuf = np.empty((B, K, Hz, Wz), np.float32)
    occ = np.empty((B, N), np.uint8)
    clear = np.empty((B, N), np.uint8)
    lib().emc2o_occlusion(B, N, C, K, _p(points, _F), _p(proj, _F), H, W, _p(vis, _U8), int(cell),
                          ctypes.c_float(margin), _p(zbuf, _F), _p(occ, _U8), _p(clear, _U8))
    return zbuf, occ, clear


def scene_route(offsets: np.ndarray, priority: Sequence[int], min_points: int = 1) -> np.ndarray:
    """Scene-level expert per frame from the dispatch offsets (Sec. 3.2)."""
    offsets = np.ascontiguousarray(offsets, np.int32)
    B, E1 = offsets.shape
    pr = np.ascontiguousarray(priority, np.uint8)
    assert len(pr) == E1 - 1
    out = np.empty(B, np.int32)
    lib().emc2o_scene_route(B, E1 - 1, _p(offsets, _I), _p(pr, _U8), int(min_points), _p(out, _I))
    return out


def rulebook(coords: np.ndarray):
    """3 x 3 x 3 submanifold rulebook of a voxel list [M, 4] (b, z, y, x): offsets [28], in, out."""
    coords = np.ascontiguousarray(coords, np.int32)
    M = coords.shape[0]
    offsets = np.empty(28, np.int32)
    rin = np.empty(27 * max(M, 1), np.int32)
    rout = np.empty(27 * max(M, 1), np.int32)
    n = lib().emc2o_rulebook(M, _p(coords, _I), _p(offsets, _I), _p(rin, _I), _p(rout, _I))
    return offsets, rin[:n].copy(), rout[:n].copy()


def bridge(w, batch: Dict[str, np.ndarray]) -> Dict[str, object]:
    """All four stages on one batch of a workload description (emc2_gen.Workload)."""
    pts, proj, feat = batch["points"], batch["proj"], batch["feat"]
    out: Dict[str, object] = {}
    for s, g in enumerate(w.grids):
        out[f"vox{s}"] = voxelize(pts, g.min, g.voxel, g.dims, g.max_points)
    g1 = w.grids[1]
    out["bev"] = bev(pts.shape[0], pts.shape[2], g1.dims[1], g1.dims[0], out["vox1"]["coords"],
                     out["vox1"]["mean"])
    uvd, mask, cam = project(pts, proj, w.img_h, w.img_w, w.min_depth)
    out["uvd"], out["vis_mask"], out["cam"] = uvd, mask, cam
    out["gathered"] = gather(uvd, cam, feat, w.feat_stride, getattr(w, "feat_offset", 0.0))
    out["expert"] = route(pts, mask, w.thresholds, w.lut)
    off, perm, pout, fout = dispatch(out["expert"], pts, out["gathered"], w.num_experts)
    out["offsets"], out["perm"], out["points_out"], out["feat_out"] = off, perm, pout, fout
    return out
