"""Workload descriptions: grids, cameras, routing tables and batch shapes.

Plain data only (no bridge arithmetic).  The five entries follow the benchmark
configurations: a tiny frame, a KITTI-shaped batch, a nuScenes-shaped batch, a
dense-urban stress frame and the throughput-sweep cells.  Distance thresholds
use the dispatcher's "near is < D, far is >= D" convention (Sec. 3.2) and, for
the nuScenes-shaped workload, the 35 m split of Sec. 4.1.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import List, Tuple


@dataclass(frozen=True)
class Grid:
    min: Tuple[float, float, float]
    voxel: Tuple[float, float, float]
    dims: Tuple[int, int, int]          # (Gx, Gy, Gz)
    max_points: int = 0                 # 0 = no cap

    @property
    def cells(self) -> int:
        return self.dims[0] * self.dims[1] * self.dims[2]


@dataclass(frozen=True)
class Camera:
    fx: float
    fy: float
    cx: float
    cy: float
    yaw_deg: float = 0.0


@dataclass(frozen=True)
class Workload:
    name: str
    config_id: int
    generator: str                      # "uniform" | "kitti" | "nuscenes" | "dense"
    B: int
    N: int
    C: int
    grids: Tuple[Grid, Grid]            # [0] fine voxels, [1] pillars
    cameras: Tuple[Camera, ...]
    img_h: int
    img_w: int
    feat_c: int
    feat_stride: int
    min_depth: float
    thresholds: Tuple[float, ...]       # ascending, metres
    num_experts: int
    lut: Tuple[Tuple[int, ...], Tuple[int, ...]]   # [visible?][distance bucket]
    xy_range: Tuple[float, float, float, float] = (0.0, 70.4, -40.0, 40.0)
    feat_offset: float = 0.0            # pixel position of texel 0 (non-zero for pooled maps)

    @property
    def K(self) -> int:
        return len(self.cameras)

    @property
    def feat_h(self) -> int:
        return -(-self.img_h // self.feat_stride)

    @property
    def feat_w(self) -> int:
        return -(-self.img_w // self.feat_stride)

    def with_shape(self, B: int, N: int) -> "Workload":
        return replace(self, B=B, N=N, name=f"{self.name}_B{B}_N{N}")


def _dims(lo, hi, v):
    """Cells along an axis; the last voxel may be partial so no in-box point is lost."""
    return int(math.ceil((hi - lo) / v - 1e-4))


def _grid(x, y, z, v, cap=0) -> Grid:
    return Grid(min=(x[0], y[0], z[0]), voxel=v,
                dims=(_dims(x[0], x[1], v[0]), _dims(y[0], y[1], v[1]), _dims(z[0], z[1], v[2])),
                max_points=cap)


_KITTI_X, _KITTI_Y, _KITTI_Z = (0.0, 70.4), (-40.0, 40.0), (-3.0, 1.0)
KITTI_GRIDS = (_grid(_KITTI_X, _KITTI_Y, _KITTI_Z, (0.05, 0.05, 0.1)),
               _grid(_KITTI_X, _KITTI_Y, _KITTI_Z, (0.16, 0.16, 4.0), cap=32))
_NUS_XY, _NUS_Z = (-51.2, 51.2), (-5.0, 3.0)
NUSCENES_GRIDS = (_grid(_NUS_XY, _NUS_XY, _NUS_Z, (0.075, 0.075, 0.2)),
                  _grid(_NUS_XY, _NUS_XY, _NUS_Z, (0.2, 0.2, 8.0), cap=32))

KITTI_CAMERA = (Camera(721.5, 721.5, 609.6, 172.9, 0.0),)
# Stand-in intrinsics (about 65 degrees horizontal field of view, so cameras
# spaced 55 degrees apart overlap and exercise the lowest-camera tie-break).
NUSCENES_CAMERAS = tuple(Camera(1260.0, 1260.0, 800.0, 450.0, yaw)
                         for yaw in (0.0, 55.0, -55.0, 110.0, -110.0, 180.0))

# Three range experts for visible points; everything outside the frustum goes
# to the LiDAR-only expert 3.
LUT_RANGE3 = ((3, 3, 3, 0, 0, 0, 0, 0), (0, 1, 2, 0, 0, 0, 0, 0))
# near-visible 0, far-visible 1, occluded/out-of-view 2, beyond 50 m 3.
LUT_NUSCENES = ((2, 2, 3, 0, 0, 0, 0, 0), (0, 1, 3, 0, 0, 0, 0, 0))


def _kitti_like(name, cid, gen, B, N) -> Workload:
    return Workload(name=name, config_id=cid, generator=gen, B=B, N=N, C=4, grids=KITTI_GRIDS,
                    cameras=KITTI_CAMERA, img_h=375, img_w=1242, feat_c=64, feat_stride=4,
                    min_depth=0.1, thresholds=(20.0, 40.0), num_experts=4, lut=LUT_RANGE3)


TINY = _kitti_like("tiny", 0, "uniform", 1, 16384)
KITTI = _kitti_like("kitti", 1, "kitti", 8, 120000)
NUSCENES = Workload(name="nuscenes", config_id=2, generator="nuscenes", B=4, N=300000, C=5,
                    grids=NUSCENES_GRIDS, cameras=NUSCENES_CAMERAS, img_h=900, img_w=1600,
                    feat_c=80, feat_stride=8, min_depth=0.1, thresholds=(35.0, 50.0),
                    num_experts=4, lut=LUT_NUSCENES, xy_range=(-51.2, 51.2, -51.2, 51.2))
DENSE = _kitti_like("dense", 3, "dense", 1, 300000)
# Sweep cells: KITTI-shaped points and grids seen through the six nuScenes-shaped cameras.
SWEEP = Workload(name="sweep", config_id=4, generator="kitti", B=1, N=16384, C=4, grids=KITTI_GRIDS,
                 cameras=NUSCENES_CAMERAS, img_h=900, img_w=1600, feat_c=80, feat_stride=8,
                 min_depth=0.1, thresholds=(35.0, 50.0), num_experts=4, lut=LUT_NUSCENES)
SWEEP_POINTS = (16384, 65536, 131072, 262144, 524288)
SWEEP_BATCH = (1, 8, 32)

WORKLOADS: List[Workload] = [TINY, KITTI, NUSCENES, DENSE, SWEEP]


def workload(config_id: int) -> Workload:
    return WORKLOADS[config_id]
