"""Seeded synthetic frames standing in for KITTI- and nuScenes-shaped sensor data.

The generators reproduce the shapes and gross statistics the benchmark
configurations ask for (ground plane with 1/r^2 areal density, car-sized boxes,
Beta(2,5) intensity, a 10-sweep time-lag channel, dense urban clutter); they do
not reproduce any dataset item.  Seed of a frame = config_id * 1000 + frame.

Only inputs are made here: points, 3x4 LiDAR-to-pixel matrices and per-camera
feature maps.  Nothing in this module voxelizes, projects, routes or sorts.
"""
from __future__ import annotations

import math
from typing import Dict, Optional, Sequence

import numpy as np

from .configs import Workload
from .rng import Stream

CAR = (3.9, 1.6, 1.56)
POLE = (0.4, 0.4, 1.8)


def frame_seed(w: Workload, frame: int) -> int:
    return w.config_id * 1000 + frame


# ----------------------------------------------------------------------------- points
def _ground(seed, n, r0, r1, z0, tag="ground"):
    s = Stream(seed, tag)
    r = r0 * np.power(r1 / r0, s.uniform(n))          # log-uniform range: areal density ~ 1/r^2
    az = s.uniform(n, -math.pi, math.pi)
    z = z0 + 0.05 * s.normal(n)
    return np.stack([r * np.cos(az), r * np.sin(az), z], axis=1)


def _boxes(seed, centres, yaws, sizes, per_box, z_base, tag="boxpts"):
    s = Stream(seed, tag)
    nb = len(centres)
    u = s.uniform(nb * per_box * 3).reshape(nb, per_box, 3)
    sizes = np.asarray(sizes, dtype=np.float64).reshape(nb, 1, 3)
    lx = (u[..., 0] - 0.5) * sizes[..., 0]
    ly = (u[..., 1] - 0.5) * sizes[..., 1]
    lz = u[..., 2] * sizes[..., 2]
    c, sn = np.cos(yaws)[:, None], np.sin(yaws)[:, None]
    x = centres[:, 0:1] + c * lx - sn * ly
    y = centres[:, 1:2] + sn * lx + c * ly
    z = z_base + lz
    return np.stack([x, y, z], axis=2).reshape(nb * per_box, 3)


def _kitti_xyz(seed, n):
    per_box = (3 * n // 10) // 20
    n_box = per_box * 20
    s = Stream(seed, "boxes")
    centres = np.stack([s.uniform(20, 5.0, 65.0), s.uniform(20, -35.0, 35.0)], axis=1)
    yaws = s.uniform(20, 0.0, math.pi)
    parts = [_ground(seed, n - n_box, 2.5, 70.4, -1.7)]
    if per_box:
        parts.append(_boxes(seed, centres, yaws, [CAR] * 20, per_box, -1.7))
    return np.concatenate(parts, axis=0)


def _nuscenes_xyz(seed, n):
    per_box = (3 * n // 10) // 40
    n_box = per_box * 40
    n_ground = n - n_box
    kept, got, rnd = [], 0, 0
    while got < n_ground:                              # rejection to the square
        g = _ground(seed, max(2 * n_ground, 1024), 1.5, 72.4, -1.84, tag=f"ground{rnd}")
        ok = (np.abs(g[:, 0]) < 51.2) & (np.abs(g[:, 1]) < 51.2)
        kept.append(g[ok])
        got += int(ok.sum())
        rnd += 1
    ground = np.concatenate(kept, axis=0)[:n_ground]
    s = Stream(seed, "boxes")
    centres = np.stack([s.uniform(40, -45.0, 45.0), s.uniform(40, -45.0, 45.0)], axis=1)
    yaws = s.uniform(40, 0.0, math.pi)
    parts = [ground]
    if per_box:
        parts.append(_boxes(seed, centres, yaws, [CAR] * 40, per_box, -1.84))
    xyz = np.concatenate(parts, axis=0)
    xyz[:, 2] = np.clip(xyz[:, 2], -5.0, 3.0)
    return xyz


def _dense_xyz(seed, n):
    per_box = (6 * n // 10) // 150
    n_box = per_box * 150
    s = Stream(seed, "boxes")
    # 100 car-sized boxes anywhere in the forward half disc of radius 25 m.
    rc = 25.0 * np.sqrt(s.uniform(100))
    ac = s.uniform(100, -math.pi / 2, math.pi / 2)
    car_c = np.stack([rc * np.cos(ac), rc * np.sin(ac)], axis=1)
    # 50 poles on distinct sites of a 2 m lattice (4 m <= r <= 25 m), so poles never overlap.
    gx, gy = np.meshgrid(np.arange(0.0, 26.0, 2.0), np.arange(-24.0, 26.0, 2.0), indexing="ij")
    sites = np.stack([gx.ravel(), gy.ravel()], axis=1)
    rr = np.hypot(sites[:, 0], sites[:, 1])
    sites = sites[(rr >= 4.0) & (rr <= 24.0)]
    pick = s.permutation(len(sites))[:50]
    pole_c = sites[pick] + s.uniform(100, -0.5, 0.5).reshape(50, 2)
    centres = np.concatenate([car_c, pole_c], axis=0)
    yaws = s.uniform(150, 0.0, math.pi)
    sizes = [CAR] * 100 + [POLE] * 50
    parts = [_ground(seed, n - n_box, 2.5, 70.4, -1.7)]
    if per_box:
        parts.append(_boxes(seed, centres, yaws, sizes, per_box, -1.7))
    return np.concatenate(parts, axis=0)


def make_points(w: Workload, frame: int) -> np.ndarray:
    """float32 [N, C]: x, y, z, intensity (and a time-lag channel when C = 5)."""
    seed, n = frame_seed(w, frame), w.N
    if w.generator == "uniform":
        s = Stream(seed, "uniform")
        x0, x1, y0, y1 = w.xy_range
        cols = [s.uniform(n, x0, x1), s.uniform(n, y0, y1), s.uniform(n, -3.0, 1.0), s.uniform(n)]
        pts = np.stack(cols, axis=1)
    else:
        xyz = {"kitti": _kitti_xyz, "nuscenes": _nuscenes_xyz, "dense": _dense_xyz}[w.generator](seed, n)
        inten = Stream(seed, "intensity").beta25(n)
        pts = np.concatenate([xyz, inten[:, None]], axis=1)
        pts = pts[Stream(seed, "shuffle").permutation(n)]   # index order != spatial order
    if w.C == 5:
        lag = 0.05 * Stream(seed, "timelag").integers(n, 10).astype(np.float64)
        pts = np.concatenate([pts, lag[:, None]], axis=1)
    assert pts.shape == (n, w.C)
    return np.ascontiguousarray(pts.astype(np.float32))


# ----------------------------------------------------------------------------- cameras
def make_projection(w: Workload) -> np.ndarray:
    """float32 [K, 3, 4], row-major: LiDAR-frame homogeneous point -> (u*d, v*d, d).

    LiDAR axes: x forward, y left, z up.  Camera axes: x right, y down, z forward.
    A camera with yaw psi looks along the LiDAR direction (cos psi, sin psi, 0);
    translation is zero.
    """
    out = np.zeros((w.K, 3, 4), dtype=np.float64)
    for k, cam in enumerate(w.cameras):
        psi = math.radians(cam.yaw_deg)
        c, s = math.cos(psi), math.sin(psi)
        xc = np.array([s, -c, 0.0])        # right  = -left', with left' = (-s, c, 0)
        yc = np.array([0.0, 0.0, -1.0])    # down
        zc = np.array([c, s, 0.0])         # forward
        out[k, 0, :3] = cam.fx * xc + cam.cx * zc
        out[k, 1, :3] = cam.fy * yc + cam.cy * zc
        out[k, 2, :3] = zc
    return out.astype(np.float32)


def make_features(w: Workload, frame: int) -> np.ndarray:
    """float32 [K, Hf, Wf, Cf], channels-last, N(0,1)."""
    n = w.K * w.feat_h * w.feat_w * w.feat_c
    f = Stream(frame_seed(w, frame), "features").normal_f32(n)
    return f.reshape(w.K, w.feat_h, w.feat_w, w.feat_c)


def make_batch(w: Workload, frames: Optional[Sequence[int]] = None,
               feature_frames: Optional[int] = None) -> Dict[str, np.ndarray]:
    """Buffers for one call: points [B,N,C], proj [B,K,3,4], feat [B,K,Hf,Wf,Cf].

    ``feature_frames`` (throughput sweeps only) makes just that many distinct
    feature maps and repeats them over the batch, to bound generation time.
    """
    frames = list(range(w.B)) if frames is None else list(frames)
    pts = np.stack([make_points(w, f) for f in frames], axis=0)
    proj = np.broadcast_to(make_projection(w), (len(frames), w.K, 3, 4)).copy()
    nf = len(frames) if feature_frames is None else min(feature_frames, len(frames))
    maps = [make_features(w, f) for f in frames[:nf]]
    feat = np.stack([maps[i % nf] for i in range(len(frames))], axis=0)
    return {"points": pts, "proj": proj, "feat": feat}
