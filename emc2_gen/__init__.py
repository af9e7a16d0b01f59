"""Seeded synthetic inputs (points, calibration, feature maps) for the EMC2 bridge.

Shared as *data* by the CPU oracle's tests and the CUDA path's tests and
benchmarks; contains none of the method's arithmetic.
"""
from .configs import (DENSE, KITTI, KITTI_GRIDS, NUSCENES_GRIDS, LUT_NUSCENES, LUT_RANGE3, NUSCENES, SWEEP, SWEEP_BATCH, SWEEP_POINTS, TINY, WORKLOADS,
                      Camera, Grid, Workload, workload)
from .frames import frame_seed, make_batch, make_features, make_points, make_projection

__all__ = ["DENSE", "KITTI", "KITTI_GRIDS", "NUSCENES_GRIDS", "LUT_NUSCENES", "LUT_RANGE3", "NUSCENES", "SWEEP", "SWEEP_BATCH", "SWEEP_POINTS", "TINY", "WORKLOADS",
           "Camera", "Grid", "Workload", "workload", "frame_seed", "make_batch", "make_features",
           "make_points", "make_projection"]
