"""Thin Python binding of libemc2_bridge.so (argument marshalling only).

Every step of the path runs inside the CUDA library; this module allocates
torch tensors for the outputs, passes ``data_ptr()`` values and the current
CUDA stream through the C ABI declared in ``include/emc2_bridge.h`` and turns
status codes into exceptions.  There is no CPU fallback: if the shared library
is missing or no CUDA device is present, construction fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, List, Optional, Sequence, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libemc2_bridge.so")

EMC2_OK = 0
EMC2_ERR_INVALID_ARG = -1
EMC2_ERR_BAD_CONFIG = -2
EMC2_ERR_CUDA = -3
EMC2_ERR_CAPACITY = -4
EMC2_ERR_TIMEOUT = -5
EMC2_ERR_INTERNAL = -6
EMC2_ERR_TOO_LARGE = -7
STATIC_SCRATCH_ENTRIES = 1 << 18

# Every symbol include/emc2_bridge.h declares.
ABI_SYMBOLS = (
    "emc2_bridge_create", "emc2_voxelize", "emc2_project_gather", "emc2_route_dispatch",
    "emc2_bridge_status", "emc2_bridge_destroy", "emc2_status_string", "emc2_bridge_last_cuda_error",
    "emc2_bridge_scratch_bytes", "emc2_bridge_kernel_kinds", "emc2_bridge_kernel_name",
    "emc2_bridge_profile_enable", "emc2_bridge_profile_read", "emc2_route_dispatch_static",
    "emc2_bridge_run", "emc2_bridge_run_host", "emc2_bridge_set_overlap", "emc2_scene_route", "emc2_pool_features",
    "emc2_features_channels_last",
    "emc2_voxel_image", "emc2_voxel_image_sampled", "emc2_occlusion", "emc2_rulebook",
    "emc2_bridge_set_tuning", "emc2_bridge_profile_timeline", "emc2_voxel_image_pooled",
)

# emc2_tuning_t
TUNE_ROW_STORE = 0
TUNE_MARK_IN_PROJECTION = 1
TUNE_DEDUP_FINE = 2
TUNE_DEDUP_PILLARS = 3
TUNE_SPLIT_BATCH = 4
TUNE_NAMES = {"row_store": TUNE_ROW_STORE, "mark_in_projection": TUNE_MARK_IN_PROJECTION,
              "dedup_fine": TUNE_DEDUP_FINE, "dedup_pillars": TUNE_DEDUP_PILLARS, "split_batch": TUNE_SPLIT_BATCH}


class Emc2Grid(ctypes.Structure):
    _fields_ = [("min", ctypes.c_float * 3), ("voxel", ctypes.c_float * 3),
                ("dims", ctypes.c_int32 * 3), ("max_points", ctypes.c_int32)]


class Emc2Config(ctypes.Structure):
    _fields_ = [("device", ctypes.c_int32), ("max_batch", ctypes.c_int32),
                ("max_points", ctypes.c_int32), ("point_floats", ctypes.c_int32),
                ("grid", Emc2Grid * 2),
                ("num_cameras", ctypes.c_int32), ("img_h", ctypes.c_int32), ("img_w", ctypes.c_int32),
                ("feat_h", ctypes.c_int32), ("feat_w", ctypes.c_int32), ("feat_c", ctypes.c_int32),
                ("feat_stride", ctypes.c_int32), ("min_depth", ctypes.c_float),
                ("num_thresholds", ctypes.c_int32), ("thresholds", ctypes.c_float * 7),
                ("num_experts", ctypes.c_int32), ("lut", (ctypes.c_uint8 * 8) * 2),
                ("feat_offset", ctypes.c_float)]


class Emc2Error(RuntimeError):
    def __init__(self, status: int, where: str, text: str):
        super().__init__(f"{where}: {text} (status {status})")
        self.status = status


_lib: Optional[ctypes.CDLL] = None


def load_library() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with paper_2507_04123_b200.build.build(); "
                           "there is no fallback path")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, P = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER
    lib.emc2_bridge_create.argtypes = [P(Emc2Config), P(vp)]
    lib.emc2_voxelize.argtypes = [vp, i32, i32, vp, P(vp), P(vp), P(vp), P(vp), P(i32), vp, vp, vp]
    lib.emc2_project_gather.argtypes = [vp, i32, i32] + [vp] * 8
    lib.emc2_route_dispatch.argtypes = [vp, i32, i32] + [vp] * 9
    lib.emc2_bridge_run.argtypes = ([vp, i32, i32, vp, vp, vp, P(vp), P(vp), P(vp), P(vp), P(i32), vp, vp]
                                    + [vp] * 4 + [vp] * 5 + [vp])
    lib.emc2_bridge_run_host.argtypes = ([vp, i32, i32] + [vp] * 6 + [P(vp), P(vp), P(vp), P(vp), P(i32), vp, vp]
                                         + [vp] * 4 + [vp] * 5 + [vp, vp, vp])
    lib.emc2_route_dispatch_static.argtypes = [P(Emc2Config), i32, i32] + [vp] * 9
    lib.emc2_bridge_status.argtypes = [vp, vp]
    lib.emc2_occlusion.argtypes = [vp, i32, i32, vp, vp, vp, i32, ctypes.c_float, vp, vp, vp, vp]
    lib.emc2_voxel_image.argtypes = [vp, i32, i32, i32] + [vp] * 8
    lib.emc2_voxel_image_sampled.argtypes = [vp, i32, i32, i32] + [vp] * 9
    lib.emc2_voxel_image_pooled.argtypes = [vp, i32, i32, i32] + [vp] * 6 + [i32, vp, vp, vp]
    lib.emc2_rulebook.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, ctypes.c_int64, vp]
    lib.emc2_pool_features.argtypes = [vp, i32, i32, vp, vp, vp]
    lib.emc2_features_channels_last.argtypes = [vp, i32, vp, vp, vp]
    lib.emc2_scene_route.argtypes = [vp, i32, vp, P(ctypes.c_uint8), i32, vp, vp]
    lib.emc2_bridge_set_overlap.argtypes = [vp, ctypes.c_int]
    lib.emc2_bridge_set_tuning.argtypes = [vp, i32, i32]
    lib.emc2_bridge_profile_timeline.argtypes = [vp, P(i32), P(ctypes.c_float), P(ctypes.c_float), i32]
    lib.emc2_bridge_destroy.argtypes = [vp]
    lib.emc2_status_string.argtypes = [ctypes.c_int]
    lib.emc2_status_string.restype = ctypes.c_char_p
    lib.emc2_bridge_last_cuda_error.argtypes = [vp]
    lib.emc2_bridge_scratch_bytes.argtypes = [vp]
    lib.emc2_bridge_scratch_bytes.restype = ctypes.c_size_t
    lib.emc2_bridge_kernel_name.argtypes = [ctypes.c_int]
    lib.emc2_bridge_kernel_name.restype = ctypes.c_char_p
    lib.emc2_bridge_profile_enable.argtypes = [vp, ctypes.c_int]
    lib.emc2_bridge_profile_read.argtypes = [vp, P(ctypes.c_int64), P(ctypes.c_double), ctypes.c_int]
    _lib = lib
    return lib


def make_config(*, device: int, max_batch: int, max_points: int, point_floats: int, grids,
                num_cameras: int, img_h: int, img_w: int, feat_h: int, feat_w: int, feat_c: int,
                feat_stride: int, min_depth: float, thresholds: Sequence[float], num_experts: int,
                lut: Sequence[Sequence[int]], feat_offset: float = 0.0) -> Emc2Config:
    """Fills an emc2_config_t.  ``grids`` is two objects with min, voxel, dims, max_points."""
    c = Emc2Config()
    c.device, c.max_batch, c.max_points, c.point_floats = device, max_batch, max_points, point_floats
    for s in range(2):
        g = grids[s]
        for d in range(3):
            c.grid[s].min[d] = g.min[d]
            c.grid[s].voxel[d] = g.voxel[d]
            c.grid[s].dims[d] = g.dims[d]
        c.grid[s].max_points = g.max_points
    c.num_cameras, c.img_h, c.img_w = num_cameras, img_h, img_w
    c.feat_h, c.feat_w, c.feat_c, c.feat_stride = feat_h, feat_w, feat_c, feat_stride
    c.min_depth = min_depth
    c.feat_offset = feat_offset
    c.num_thresholds = len(thresholds)
    for t, v in enumerate(thresholds):
        c.thresholds[t] = v
    c.num_experts = num_experts
    for v in range(2):
        row = list(lut[v])[:8]
        for d, e in enumerate(row):
            c.lut[v][d] = e
    return c


def config_from_workload(w, device: int = 0, max_batch: Optional[int] = None,
                         max_points: Optional[int] = None) -> Emc2Config:
    """emc2_config_t for a workload description with the fields of emc2_gen.Workload."""
    return make_config(device=device, max_batch=max_batch or w.B, max_points=max_points or w.N,
                       point_floats=w.C, grids=w.grids, num_cameras=w.K, img_h=w.img_h, img_w=w.img_w,
                       feat_h=w.feat_h, feat_w=w.feat_w, feat_c=w.feat_c, feat_stride=w.feat_stride,
                       min_depth=w.min_depth, thresholds=w.thresholds, num_experts=w.num_experts,
                       lut=w.lut, feat_offset=getattr(w, "feat_offset", 0.0))


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _check(t: torch.Tensor, dtype, shape, name: str, device) -> None:
    if t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous() or t.device != device:
        raise ValueError(f"{name}: expected contiguous {dtype} {tuple(shape)} on {device}, "
                         f"got {t.dtype} {tuple(t.shape)} on {t.device}")


def route_dispatch_static(config: Emc2Config, points: torch.Tensor, vis_mask: torch.Tensor,
                          gathered: torch.Tensor, out: Dict[str, torch.Tensor]) -> Dict[str, torch.Tensor]:
    """emc2_route_dispatch_static: stages 3 and 4 without a handle and without any allocation.

    For hosts that may not allocate device memory where they dispatch (an engine plug-in confined
    to the engine's pool, a real-time loop).  The library's only scratch is a fixed array inside
    its image, so the call is limited to B * ceil(N / 256) * num_experts <= STATIC_SCRATCH_ENTRIES
    and calls that can overlap on one device must be ordered by the caller.  ``out`` must hold the
    five preallocated output tensors of :meth:`Bridge.route_dispatch`; nothing is allocated here.
    """
    lib = load_library()
    B, N, C = points.shape
    dev = points.device
    if dev.type != "cuda" or dev.index != config.device:
        raise ValueError(f"points live on {dev}, the configuration names CUDA device {config.device}")
    _check(points, torch.float32, (B, N, config.point_floats), "points", dev)
    _check(vis_mask, torch.uint8, (B, N), "vis_mask", dev)
    _check(gathered, torch.float32, (B, N, config.feat_c), "gathered", dev)
    _check(out["expert"], torch.uint8, (B, N), "expert", dev)
    _check(out["offsets"], torch.int32, (B, config.num_experts + 1), "offsets", dev)
    _check(out["perm"], torch.int32, (B, N), "perm", dev)
    _check(out["points_out"], torch.float32, (B, N, C), "points_out", dev)
    _check(out["feat_out"], torch.float32, (B, N, config.feat_c), "feat_out", dev)
    rc = lib.emc2_route_dispatch_static(ctypes.byref(config), B, N, points.data_ptr(), vis_mask.data_ptr(),
                                        gathered.data_ptr(), out["expert"].data_ptr(),
                                        out["offsets"].data_ptr(), out["perm"].data_ptr(),
                                        out["points_out"].data_ptr(), out["feat_out"].data_ptr(),
                                        torch.cuda.current_stream(dev).cuda_stream)
    if rc != EMC2_OK:
        raise Emc2Error(rc, "emc2_route_dispatch_static", lib.emc2_status_string(rc).decode())
    return out


class Bridge:
    """One emc2_bridge_t handle.  Methods mirror the C entry points."""

    def __init__(self, config: Emc2Config):
        if not torch.cuda.is_available():
            raise RuntimeError("emc2 bridge needs a CUDA device; there is no CPU path")
        self.lib = load_library()
        self.cfg = config
        self.device = torch.device("cuda", config.device)
        self._h = ctypes.c_void_p()
        rc = self.lib.emc2_bridge_create(ctypes.byref(config), ctypes.byref(self._h))
        self._raise(rc, "emc2_bridge_create")

    # ------------------------------------------------------------------ helpers
    def _raise(self, rc: int, where: str) -> None:
        if rc != EMC2_OK:
            raise Emc2Error(rc, where, self.lib.emc2_status_string(rc).decode())

    def _stream(self) -> int:
        return torch.cuda.current_stream(self.device).cuda_stream

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            torch.cuda.synchronize(self.device)
            self.lib.emc2_bridge_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def scratch_bytes(self) -> int:
        return int(self.lib.emc2_bridge_scratch_bytes(self._h))

    # ------------------------------------------------------------------ stage calls
    def voxelize(self, points: torch.Tensor, capacity: Optional[Sequence[int]] = None,
                 want_point_voxel: bool = True, want_bev: bool = True,
                 out: Optional[Dict[str, object]] = None) -> Dict[str, object]:
        """emc2_voxelize.  Returns device tensors; rows past num_voxels[s] are unspecified."""
        B, N, C = points.shape
        _check(points, torch.float32, (B, N, self.cfg.point_floats), "points", self.device)
        cap = list(capacity) if capacity is not None else [B * N, B * N]
        dev = self.device
        if out is None:
            out = {
                "coords": [torch.empty((max(cap[s], 1), 4), dtype=torch.int32, device=dev) for s in range(2)],
                "counts": [torch.empty((max(cap[s], 1),), dtype=torch.int32, device=dev) for s in range(2)],
                "mean": [torch.empty((max(cap[s], 1), C), dtype=torch.float32, device=dev) for s in range(2)],
                "point_voxel": [torch.empty((B, N), dtype=torch.int32, device=dev) for _ in range(2)]
                if want_point_voxel else None,
                "num_voxels": torch.empty((2,), dtype=torch.int32, device=dev),
                "bev": torch.empty((B, C, self.cfg.grid[1].dims[1], self.cfg.grid[1].dims[0]),
                                   dtype=torch.float32, device=dev) if want_bev else None,
            }
        arr = ctypes.c_void_p * 2
        pv = out["point_voxel"]
        rc = self.lib.emc2_voxelize(
            self._h, B, N, points.data_ptr(),
            arr(*[t.data_ptr() for t in out["coords"]]), arr(*[t.data_ptr() for t in out["counts"]]),
            arr(*[t.data_ptr() for t in out["mean"]]),
            arr(*[t.data_ptr() for t in pv]) if pv is not None else None,
            (ctypes.c_int32 * 2)(*cap), out["num_voxels"].data_ptr(), _ptr(out["bev"]), self._stream())
        self._raise(rc, "emc2_voxelize")
        return out

    def project_gather(self, points: torch.Tensor, proj: torch.Tensor, feat: torch.Tensor,
                       out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
        """emc2_project_gather."""
        B, N, C = points.shape
        c = self.cfg
        _check(points, torch.float32, (B, N, c.point_floats), "points", self.device)
        _check(proj, torch.float32, (B, c.num_cameras, 3, 4), "proj", self.device)
        _check(feat, torch.float32, (B, c.num_cameras, c.feat_h, c.feat_w, c.feat_c), "feat", self.device)
        if out is None:
            dev = self.device
            out = {"uvd": torch.empty((B, N, 3), dtype=torch.float32, device=dev),
                   "vis_mask": torch.empty((B, N), dtype=torch.uint8, device=dev),
                   "cam": torch.empty((B, N), dtype=torch.int8, device=dev),
                   "gathered": torch.empty((B, N, c.feat_c), dtype=torch.float32, device=dev)}
        rc = self.lib.emc2_project_gather(self._h, B, N, points.data_ptr(), proj.data_ptr(), feat.data_ptr(),
                                          out["uvd"].data_ptr(), out["vis_mask"].data_ptr(),
                                          out["cam"].data_ptr(), out["gathered"].data_ptr(), self._stream())
        self._raise(rc, "emc2_project_gather")
        return out

    def route_dispatch(self, points: torch.Tensor, vis_mask: torch.Tensor, gathered: torch.Tensor,
                       out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
        """emc2_route_dispatch."""
        B, N, C = points.shape
        c = self.cfg
        _check(points, torch.float32, (B, N, c.point_floats), "points", self.device)
        _check(vis_mask, torch.uint8, (B, N), "vis_mask", self.device)
        _check(gathered, torch.float32, (B, N, c.feat_c), "gathered", self.device)
        if out is None:
            dev = self.device
            out = {"expert": torch.empty((B, N), dtype=torch.uint8, device=dev),
                   "offsets": torch.empty((B, c.num_experts + 1), dtype=torch.int32, device=dev),
                   "perm": torch.empty((B, N), dtype=torch.int32, device=dev),
                   "points_out": torch.empty_like(points),
                   "feat_out": torch.empty_like(gathered)}
        rc = self.lib.emc2_route_dispatch(self._h, B, N, points.data_ptr(), vis_mask.data_ptr(),
                                          gathered.data_ptr(), out["expert"].data_ptr(),
                                          out["offsets"].data_ptr(), out["perm"].data_ptr(),
                                          out["points_out"].data_ptr(), out["feat_out"].data_ptr(),
                                          self._stream())
        self._raise(rc, "emc2_route_dispatch")
        return out

    def voxel_image(self, vox: Dict[str, object], scale: int, vis_mask: torch.Tensor, gathered: torch.Tensor,
                    out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
        """emc2_voxel_image for one scale of a :meth:`voxelize` result (needs its point_voxel)."""
        B, N = vis_mask.shape
        c = self.cfg
        pv = vox["point_voxel"][scale]
        counts = vox["counts"][scale]
        cap = int(counts.shape[0])
        _check(pv, torch.int32, (B, N), "point_voxel", self.device)
        _check(vis_mask, torch.uint8, (B, N), "vis_mask", self.device)
        _check(gathered, torch.float32, (B, N, c.feat_c), "gathered", self.device)
        if out is None:
            out = {"vox_img": torch.empty((cap, c.feat_c), dtype=torch.float32, device=self.device),
                   "vox_img_count": torch.empty((cap,), dtype=torch.int32, device=self.device)}
        nv = vox["num_voxels"]
        rc = self.lib.emc2_voxel_image(self._h, B, N, cap, pv.data_ptr(), counts.data_ptr(),
                                       nv.data_ptr() + 4 * scale, vis_mask.data_ptr(), gathered.data_ptr(),
                                       out["vox_img"].data_ptr(), out["vox_img_count"].data_ptr(), self._stream())
        self._raise(rc, "emc2_voxel_image")
        return out

    def voxel_image_sampled(self, vox: Dict[str, object], scale: int, uvd: torch.Tensor, cam: torch.Tensor,
                            feat: torch.Tensor, out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
        """emc2_voxel_image_sampled: per-voxel image features blended straight from the feature maps."""
        B, N = cam.shape
        c = self.cfg
        pv = vox["point_voxel"][scale]
        counts = vox["counts"][scale]
        cap = int(counts.shape[0])
        _check(pv, torch.int32, (B, N), "point_voxel", self.device)
        _check(uvd, torch.float32, (B, N, 3), "uvd", self.device)
        _check(cam, torch.int8, (B, N), "cam", self.device)
        _check(feat, torch.float32, (B, c.num_cameras, c.feat_h, c.feat_w, c.feat_c), "feat", self.device)
        if out is None:
            out = {"vox_img": torch.empty((cap, c.feat_c), dtype=torch.float32, device=self.device),
                   "vox_img_count": torch.empty((cap,), dtype=torch.int32, device=self.device)}
        nv = vox["num_voxels"]
        rc = self.lib.emc2_voxel_image_sampled(self._h, B, N, cap, pv.data_ptr(), counts.data_ptr(),
                                               nv.data_ptr() + 4 * scale, uvd.data_ptr(), cam.data_ptr(),
                                               feat.data_ptr(), out["vox_img"].data_ptr(),
                                               out["vox_img_count"].data_ptr(), self._stream())
        self._raise(rc, "emc2_voxel_image_sampled")
        return out

    def voxel_image_pooled(self, vox: Dict[str, object], scale: int, uvd: torch.Tensor, cam: torch.Tensor,
                           feat: torch.Tensor, p: int, out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
        """emc2_voxel_image_pooled: per-voxel image features from p x p window means of the unpooled maps."""
        B, N = cam.shape
        c = self.cfg
        pv = vox["point_voxel"][scale]
        counts = vox["counts"][scale]
        cap = int(counts.shape[0])
        _check(pv, torch.int32, (B, N), "point_voxel", self.device)
        _check(uvd, torch.float32, (B, N, 3), "uvd", self.device)
        _check(cam, torch.int8, (B, N), "cam", self.device)
        _check(feat, torch.float32, (B, c.num_cameras, c.feat_h, c.feat_w, c.feat_c), "feat", self.device)
        if out is None:
            out = {"vox_img": torch.empty((cap, c.feat_c), dtype=torch.float32, device=self.device),
                   "vox_img_count": torch.empty((cap,), dtype=torch.int32, device=self.device)}
        nv = vox["num_voxels"]
        rc = self.lib.emc2_voxel_image_pooled(self._h, B, N, cap, pv.data_ptr(), counts.data_ptr(),
                                              nv.data_ptr() + 4 * scale, uvd.data_ptr(), cam.data_ptr(),
                                              feat.data_ptr(), int(p), out["vox_img"].data_ptr(),
                                              out["vox_img_count"].data_ptr(), self._stream())
        self._raise(rc, "emc2_voxel_image_pooled")
        return out

    def rulebook(self, vox: Dict[str, object], scale: int, pair_capacity: Optional[int] = None,
                 out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
        """emc2_rulebook for one scale of a :meth:`voxelize` result: offsets [28], rule_in, rule_out."""
        coords = vox["coords"][scale]
        cap = int(coords.shape[0])
        _check(coords, torch.int32, (cap, 4), "coords", self.device)
        if out is None:
            pairs = 27 * cap if pair_capacity is None else int(pair_capacity)
            out = {"offsets": torch.empty((28,), dtype=torch.int32, device=self.device),
                   "rule_in": torch.empty((pairs,), dtype=torch.int32, device=self.device),
                   "rule_out": torch.empty((pairs,), dtype=torch.int32, device=self.device)}
        pairs = int(out["rule_in"].shape[0])
        _check(out["offsets"], torch.int32, (28,), "offsets", self.device)
        _check(out["rule_out"], torch.int32, (pairs,), "rule_out", self.device)
        nv = vox["num_voxels"]
        rc = self.lib.emc2_rulebook(self._h, int(scale), cap, coords.data_ptr(), nv.data_ptr() + 4 * scale,
                                    out["offsets"].data_ptr(), out["rule_in"].data_ptr(),
                                    out["rule_out"].data_ptr(), pairs, self._stream())
        self._raise(rc, "emc2_rulebook")
        return out

    def occlusion(self, points: torch.Tensor, proj: torch.Tensor, vis_mask: torch.Tensor, cell: int,
                  margin: float, out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
        """emc2_occlusion: depth buffer per camera cell, occluded bits, mask of clear views."""
        B, N, C = points.shape
        c = self.cfg
        _check(points, torch.float32, (B, N, c.point_floats), "points", self.device)
        _check(proj, torch.float32, (B, c.num_cameras, 3, 4), "proj", self.device)
        _check(vis_mask, torch.uint8, (B, N), "vis_mask", self.device)
        if out is None:
            shape = (B, c.num_cameras, -(-c.img_h // cell), -(-c.img_w // cell))
            out = {"zbuf": torch.empty(shape, dtype=torch.float32, device=self.device),
                   "occ_mask": torch.empty((B, N), dtype=torch.uint8, device=self.device),
                   "clear_mask": torch.empty((B, N), dtype=torch.uint8, device=self.device)}
        rc = self.lib.emc2_occlusion(self._h, B, N, points.data_ptr(), proj.data_ptr(), vis_mask.data_ptr(),
                                     int(cell), float(margin), out["zbuf"].data_ptr(), out["occ_mask"].data_ptr(),
                                     out["clear_mask"].data_ptr(), self._stream())
        self._raise(rc, "emc2_occlusion")
        return out

    def features_channels_last(self, planar: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """emc2_features_channels_last: [B,K,Cf,Hf,Wf] maps copied into the [B,K,Hf,Wf,Cf] layout."""
        c = self.cfg
        B = planar.shape[0]
        _check(planar, torch.float32, (B, c.num_cameras, c.feat_c, c.feat_h, c.feat_w), "planar", self.device)
        shape = (B, c.num_cameras, c.feat_h, c.feat_w, c.feat_c)
        if out is None:
            out = torch.empty(shape, dtype=torch.float32, device=self.device)
        _check(out, torch.float32, shape, "feat", self.device)
        rc = self.lib.emc2_features_channels_last(self._h, B, planar.data_ptr(), out.data_ptr(), self._stream())
        self._raise(rc, "emc2_features_channels_last")
        return out

    def pool_features(self, feat: torch.Tensor, p: int, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """emc2_pool_features: p x p average pooling of the handle's feature maps."""
        c = self.cfg
        B = feat.shape[0]
        _check(feat, torch.float32, (B, c.num_cameras, c.feat_h, c.feat_w, c.feat_c), "feat", self.device)
        shape = (B, c.num_cameras, -(-c.feat_h // p), -(-c.feat_w // p), c.feat_c)
        if out is None:
            out = torch.empty(shape, dtype=torch.float32, device=self.device)
        _check(out, torch.float32, shape, "pooled", self.device)
        rc = self.lib.emc2_pool_features(self._h, B, int(p), feat.data_ptr(), out.data_ptr(), self._stream())
        self._raise(rc, "emc2_pool_features")
        return out

    def scene_route(self, offsets: torch.Tensor, priority: Sequence[int], min_points: int = 1,
                    out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """emc2_scene_route: one expert per frame from the dispatch offsets."""
        B = offsets.shape[0]
        _check(offsets, torch.int32, (B, self.cfg.num_experts + 1), "offsets", self.device)
        if len(priority) != self.cfg.num_experts:
            raise ValueError("priority needs one entry per expert")
        if out is None:
            out = torch.empty((B,), dtype=torch.int32, device=self.device)
        pr = (ctypes.c_uint8 * len(priority))(*priority)
        rc = self.lib.emc2_scene_route(self._h, B, offsets.data_ptr(), pr, int(min_points), out.data_ptr(),
                                       self._stream())
        self._raise(rc, "emc2_scene_route")
        return out

    def set_overlap(self, enable: bool) -> None:
        """emc2_bridge_set_overlap: stage 1 of :meth:`run` beside stages 2 - 4 (default) or after them."""
        self._raise(self.lib.emc2_bridge_set_overlap(self._h, int(enable)), "emc2_bridge_set_overlap")

    def set_tuning(self, knob, value: int) -> None:
        """emc2_bridge_set_tuning: ``knob`` is an emc2_tuning_t value or its name in TUNE_NAMES."""
        k = TUNE_NAMES[knob] if isinstance(knob, str) else int(knob)
        self._raise(self.lib.emc2_bridge_set_tuning(self._h, k, int(value)), "emc2_bridge_set_tuning")

    def status(self, raise_on_error: bool = True) -> int:
        """emc2_bridge_status: waits for the current stream, returns the sticky device status."""
        rc = self.lib.emc2_bridge_status(self._h, self._stream())
        if raise_on_error:
            self._raise(rc, "emc2_bridge_status")
        return rc

    # ------------------------------------------------------------------ whole path
    def _alloc_vox(self, B, N, C, cap, want_point_voxel=True, want_bev=True):
        dev = self.device
        return {
            "coords": [torch.empty((max(cap[s], 1), 4), dtype=torch.int32, device=dev) for s in range(2)],
            "counts": [torch.empty((max(cap[s], 1),), dtype=torch.int32, device=dev) for s in range(2)],
            "mean": [torch.empty((max(cap[s], 1), C), dtype=torch.float32, device=dev) for s in range(2)],
            "point_voxel": [torch.empty((B, N), dtype=torch.int32, device=dev) for _ in range(2)]
            if want_point_voxel else None,
            "num_voxels": torch.empty((2,), dtype=torch.int32, device=dev),
            "bev": torch.empty((B, C, self.cfg.grid[1].dims[1], self.cfg.grid[1].dims[0]),
                               dtype=torch.float32, device=dev) if want_bev else None,
        }

    def run_staged(self, points: torch.Tensor, proj: torch.Tensor, feat: torch.Tensor,
                   bufs: Optional[Dict[str, object]] = None) -> Dict[str, object]:
        """The three stage calls back to back on the current stream (no host sync)."""
        bufs = bufs if bufs is not None else {}
        bufs["vox"] = self.voxelize(points, out=bufs.get("vox"))
        bufs["pg"] = self.project_gather(points, proj, feat, out=bufs.get("pg"))
        pg = bufs["pg"]
        bufs["rd"] = self.route_dispatch(points, pg["vis_mask"], pg["gathered"], out=bufs.get("rd"))
        return bufs

    def run(self, points: torch.Tensor, proj: torch.Tensor, feat: torch.Tensor,
            bufs: Optional[Dict[str, object]] = None) -> Dict[str, object]:
        """emc2_bridge_run: all stages in one call; same outputs as :meth:`run_staged`.  With
        ``bufs["pg"]["gathered"] = None`` the rows in point order are not stored."""
        B, N, C = points.shape
        c = self.cfg
        _check(points, torch.float32, (B, N, c.point_floats), "points", self.device)
        _check(proj, torch.float32, (B, c.num_cameras, 3, 4), "proj", self.device)
        _check(feat, torch.float32, (B, c.num_cameras, c.feat_h, c.feat_w, c.feat_c), "feat", self.device)
        if bufs is None:
            dev = self.device
            bufs = {"vox": self._alloc_vox(B, N, C, [B * N, B * N]),
                    "pg": {"uvd": torch.empty((B, N, 3), dtype=torch.float32, device=dev),
                           "vis_mask": torch.empty((B, N), dtype=torch.uint8, device=dev),
                           "cam": torch.empty((B, N), dtype=torch.int8, device=dev),
                           "gathered": torch.empty((B, N, c.feat_c), dtype=torch.float32, device=dev)},
                    "rd": {"expert": torch.empty((B, N), dtype=torch.uint8, device=dev),
                           "offsets": torch.empty((B, c.num_experts + 1), dtype=torch.int32, device=dev),
                           "perm": torch.empty((B, N), dtype=torch.int32, device=dev),
                           "points_out": torch.empty_like(points),
                           "feat_out": torch.empty((B, N, c.feat_c), dtype=torch.float32, device=dev)}}
        vox, pg, rd = bufs["vox"], bufs["pg"], bufs["rd"]
        arr = ctypes.c_void_p * 2
        pv = vox["point_voxel"]
        cap = [int(vox["coords"][s].shape[0]) for s in range(2)]
        rc = self.lib.emc2_bridge_run(
            self._h, B, N, points.data_ptr(), proj.data_ptr(), feat.data_ptr(),
            arr(*[t.data_ptr() for t in vox["coords"]]), arr(*[t.data_ptr() for t in vox["counts"]]),
            arr(*[t.data_ptr() for t in vox["mean"]]),
            arr(*[t.data_ptr() for t in pv]) if pv is not None else None,
            (ctypes.c_int32 * 2)(*cap), vox["num_voxels"].data_ptr(), _ptr(vox["bev"]),
            pg["uvd"].data_ptr(), pg["vis_mask"].data_ptr(), pg["cam"].data_ptr(), _ptr(pg.get("gathered")),
            rd["expert"].data_ptr(), rd["offsets"].data_ptr(), rd["perm"].data_ptr(),
            rd["points_out"].data_ptr(), rd["feat_out"].data_ptr(), self._stream())
        self._raise(rc, "emc2_bridge_run")
        return bufs

    def run_host(self, host: Dict[str, torch.Tensor], staging: Dict[str, torch.Tensor], bufs: Dict[str, object],
                 h_offsets: Optional[torch.Tensor] = None, h_num_voxels: Optional[torch.Tensor] = None) -> Dict[str, object]:
        """emc2_bridge_run_host: host tensors ``points, proj, feat`` are copied into the device tensors of
        ``staging``, the whole bridge runs into ``bufs`` (as :meth:`run` returns them), offsets and voxel
        counts are copied to the host tensors given.  Everything is only enqueued on the current stream."""
        c = self.cfg
        B, N, C = host["points"].shape
        shapes = {"points": (B, N, c.point_floats), "proj": (B, c.num_cameras, 3, 4),
                  "feat": (B, c.num_cameras, c.feat_h, c.feat_w, c.feat_c)}
        for k, shp in shapes.items():
            _check(staging[k], torch.float32, shp, "staging " + k, self.device)
            t = host[k]
            if t.device.type != "cpu" or t.dtype != torch.float32 or tuple(t.shape) != shp or not t.is_contiguous():
                raise ValueError(f"host {k}: need a contiguous float32 CPU tensor of shape {shp}")
        for t, shp, name in ((h_offsets, (B, c.num_experts + 1), "h_offsets"), (h_num_voxels, (2,), "h_num_voxels")):
            if t is not None and (t.device.type != "cpu" or t.dtype != torch.int32 or tuple(t.shape) != shp
                                  or not t.is_contiguous()):
                raise ValueError(f"{name}: need a contiguous int32 CPU tensor of shape {shp}")
        vox, pg, rd = bufs["vox"], bufs["pg"], bufs["rd"]
        arr = ctypes.c_void_p * 2
        pv = vox["point_voxel"]
        cap = [int(vox["coords"][s].shape[0]) for s in range(2)]
        rc = self.lib.emc2_bridge_run_host(
            self._h, B, N, host["points"].data_ptr(), host["proj"].data_ptr(), host["feat"].data_ptr(),
            staging["points"].data_ptr(), staging["proj"].data_ptr(), staging["feat"].data_ptr(),
            arr(*[t.data_ptr() for t in vox["coords"]]), arr(*[t.data_ptr() for t in vox["counts"]]),
            arr(*[t.data_ptr() for t in vox["mean"]]),
            arr(*[t.data_ptr() for t in pv]) if pv is not None else None,
            (ctypes.c_int32 * 2)(*cap), vox["num_voxels"].data_ptr(), _ptr(vox["bev"]),
            pg["uvd"].data_ptr(), pg["vis_mask"].data_ptr(), pg["cam"].data_ptr(), _ptr(pg.get("gathered")),
            rd["expert"].data_ptr(), rd["offsets"].data_ptr(), rd["perm"].data_ptr(),
            rd["points_out"].data_ptr(), rd["feat_out"].data_ptr(),
            h_offsets.data_ptr() if h_offsets is not None else None,
            h_num_voxels.data_ptr() if h_num_voxels is not None else None, self._stream())
        self._raise(rc, "emc2_bridge_run_host")
        return bufs

    # ------------------------------------------------------------------ measurement aids
    def kernel_names(self) -> List[str]:
        n = self.lib.emc2_bridge_kernel_kinds()
        return [self.lib.emc2_bridge_kernel_name(k).decode() for k in range(n)]

    def profile_enable(self, enable: bool) -> None:
        self._raise(self.lib.emc2_bridge_profile_enable(self._h, int(enable)), "emc2_bridge_profile_enable")

    def profile_read(self, reset: bool = True) -> Dict[str, Tuple[int, float]]:
        n = self.lib.emc2_bridge_kernel_kinds()
        launches = (ctypes.c_int64 * n)()
        ms = (ctypes.c_double * n)()
        self._raise(self.lib.emc2_bridge_profile_read(self._h, launches, ms, int(reset)),
                    "emc2_bridge_profile_read")
        return {name: (int(launches[k]), float(ms[k])) for k, name in enumerate(self.kernel_names())}

    def profile_timeline(self, capacity: int = 4096) -> List[Tuple[str, float, float]]:
        """emc2_bridge_profile_timeline: (kernel, start ms, end ms) of the launches recorded since the last read."""
        kinds = (ctypes.c_int32 * capacity)()
        t0 = (ctypes.c_float * capacity)()
        t1 = (ctypes.c_float * capacity)()
        n = self.lib.emc2_bridge_profile_timeline(self._h, kinds, t0, t1, capacity)
        if n < 0:
            self._raise(n, "emc2_bridge_profile_timeline")
        names = self.kernel_names()
        return [(names[kinds[i]], float(t0[i]), float(t1[i])) for i in range(n)]
