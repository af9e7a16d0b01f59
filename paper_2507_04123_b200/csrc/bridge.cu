// Handle management and the extern "C" entry points of the bridge library.
#include <cmath>
#include <cstring>
#include <new>

#include "bridge_internal.cuh"

namespace emc2 {

static const char* const kKernelNames[K_KINDS] = {
    "vox_mark", "vox_count", "vox_prefix", "vox_rank", "vox_accum", "vox_over_find", "vox_over_fill", "vox_finalize", "arm_keys", "arm_sort", "arm_hash", "arm_rank",
    "project_gather", "project_route", "gather_scatter", "route_hist", "route_scan", "dispatch_scatter", "scene_route", "pool_features",
    "vif_scan", "vif_fill", "vif_mean", "vif_sample", "occl_fill", "occl_splat", "occl_test",
    "channels_last", "rb_mark", "rb_count", "rb_scan", "rb_fill", "rb_clear"};

int check_cuda(emc2_bridge* h, cudaError_t e) {
    if (e == cudaSuccess) return EMC2_OK;
    if (h) h->last_cuda_error = (int)e;
    return EMC2_ERR_CUDA;
}

LaunchScope::LaunchScope(emc2_bridge* h_, int kind_, cudaStream_t st_) : h(h_), kind(kind_), st(st_) {
    h->launches[kind] += 1;
    if (!h->profiling) return;
    for (cudaEvent_t* e : {&a, &b}) {
        if (!h->event_pool.empty()) {
            *e = h->event_pool.back();
            h->event_pool.pop_back();
        } else if (cudaEventCreate(e) != cudaSuccess) {
            *e = nullptr;
        }
    }
    if (a) cudaEventRecord(a, st);
}

LaunchScope::~LaunchScope() {
    if (!h->profiling || !a || !b) return;
    cudaEventRecord(b, st);
    h->recs.push_back({kind, a, b});
}

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() {
        int cur;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

int validate(const emc2_config_t& c) {
    if (c.device < 0) return EMC2_ERR_BAD_CONFIG;
    if (c.max_batch < 1 || c.max_batch > EMC2_MAX_BATCH) return EMC2_ERR_BAD_CONFIG;
    if (c.max_points < 1) return EMC2_ERR_BAD_CONFIG;
    // Per-voxel point counts are accumulated in fp32, which is exact up to 2^24.
    if ((int64_t)c.max_batch * c.max_points > (int64_t)1 << 24) return EMC2_ERR_BAD_CONFIG;
    if (c.point_floats != 4 && c.point_floats != 5) return EMC2_ERR_BAD_CONFIG;
    for (int s = 0; s < 2; ++s) {
        const emc2_grid_t& g = c.grid[s];
        uint64_t cells = 1;
        for (int d = 0; d < 3; ++d) {
            if (!(g.voxel[d] > 0.0f) || !std::isfinite(g.voxel[d]) || !std::isfinite(g.min[d]))
                return EMC2_ERR_BAD_CONFIG;
            if (g.dims[d] < 1 || g.dims[d] > (1 << 24)) return EMC2_ERR_BAD_CONFIG;
            cells *= (uint64_t)g.dims[d];
            if (cells > 0xFFFFFFFFull) return EMC2_ERR_BAD_CONFIG;
        }
        if (cells * (uint64_t)c.max_batch > 0xFFFFFF00ull) return EMC2_ERR_BAD_CONFIG;
        if (g.max_points < 0) return EMC2_ERR_BAD_CONFIG;
    }
    if (c.grid[1].dims[2] != 1) return EMC2_ERR_BAD_CONFIG;
    if (c.num_cameras < 1 || c.num_cameras > EMC2_MAX_CAMERAS) return EMC2_ERR_BAD_CONFIG;
    if (c.img_h < 1 || c.img_w < 1 || c.feat_h < 1 || c.feat_w < 1) return EMC2_ERR_BAD_CONFIG;
    if (c.feat_c < 4 || (c.feat_c & 3)) return EMC2_ERR_BAD_CONFIG;
    if (!is_pow2(c.feat_stride)) return EMC2_ERR_BAD_CONFIG;
    // Every visible pixel must fall inside the map: (dim - 1) / stride <= feat_dim - 1.
    if ((c.img_h - 1) / c.feat_stride > c.feat_h - 1 || (c.img_w - 1) / c.feat_stride > c.feat_w - 1)
        return EMC2_ERR_BAD_CONFIG;
    // Tap addresses are 32-bit float4 indices into the feature buffer.
    if ((uint64_t)c.max_batch * c.num_cameras * c.feat_h * c.feat_w * (uint64_t)(c.feat_c / 4) > 0xFFFFFFF0ull)
        return EMC2_ERR_BAD_CONFIG;
    if (!(c.min_depth >= 0.0f)) return EMC2_ERR_BAD_CONFIG;
    if (!(c.feat_offset >= 0.0f) || !std::isfinite(c.feat_offset)) return EMC2_ERR_BAD_CONFIG;
    if (c.num_thresholds < 0 || c.num_thresholds > EMC2_MAX_THRESHOLDS) return EMC2_ERR_BAD_CONFIG;
    for (int t = 0; t < c.num_thresholds; ++t) {
        if (!(c.thresholds[t] >= 0.0f) || !std::isfinite(c.thresholds[t])) return EMC2_ERR_BAD_CONFIG;
        if (t && !(c.thresholds[t] >= c.thresholds[t - 1])) return EMC2_ERR_BAD_CONFIG;
    }
    if (c.num_experts < 1 || c.num_experts > EMC2_MAX_EXPERTS) return EMC2_ERR_BAD_CONFIG;
    for (int v = 0; v < 2; ++v)
        for (int d = 0; d <= c.num_thresholds; ++d)
            if (c.lut[v][d] >= c.num_experts) return EMC2_ERR_BAD_CONFIG;
    return EMC2_OK;
}

struct SlabPlan {
    size_t off = 0;
    size_t take(size_t bytes) {
        const size_t o = off;
        off += (bytes + 255) & ~(size_t)255;
        return o;
    }
};

}  // namespace
}  // namespace emc2

using namespace emc2;

extern "C" {

int emc2_bridge_create(const emc2_config_t* config, emc2_bridge_t** out) {
    if (!config || !out) return EMC2_ERR_INVALID_ARG;
    *out = nullptr;
    int rc = validate(*config);
    if (rc != EMC2_OK) return rc;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || config->device >= ndev) return EMC2_ERR_CUDA;
    emc2_bridge* h = new (std::nothrow) emc2_bridge();
    if (!h) return EMC2_ERR_INTERNAL;
    h->cfg = *config;
    DeviceGuard guard(config->device);
    if (!guard.ok) { delete h; return EMC2_ERR_CUDA; }

    const emc2_config_t& c = h->cfg;
    const size_t maxpts = (size_t)c.max_batch * c.max_points;
    for (int t = 0; t < EMC2_MAX_THRESHOLDS; ++t)
        h->thr2[t] = t < c.num_thresholds ? c.thresholds[t] * c.thresholds[t] : 0.0f;

    if (cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, config->device) != cudaSuccess ||
        h->num_sms < 1) { delete h; return EMC2_ERR_CUDA; }
    h->vif_scan_blocks = voxel_image_scan_max_blocks();
    if (h->vif_scan_blocks < 1) { delete h; return EMC2_ERR_CUDA; }

    // Plan the slab: everything the stage calls need, allocated once.
    SlabPlan plan;
    size_t o_store[2], o_flag[2], o_acc[2], o_cl[2], o_ovf[2][5], o_tot[2];
    for (int s = 0; s < 2; ++s) {
        ScaleDev& d = h->scale[s];
        const emc2_grid_t& g = c.grid[s];
        for (int k = 0; k < 3; ++k) {
            d.mn[k] = g.min[k]; d.vs[k] = g.voxel[k]; d.dims[k] = g.dims[k];
            d.div[k] = make_fast_div((uint32_t)g.dims[k]);
        }
        d.cap = g.max_points;
        d.design = 0;
        d.point_rank = nullptr;
        d.cells = (uint32_t)((uint64_t)g.dims[0] * g.dims[1] * g.dims[2]);
        const uint64_t total_cells = (uint64_t)d.cells * c.max_batch;
        d.mode = total_cells <= (uint64_t)kMaxTableCells ? MODE_TABLE : MODE_BITMAP;
        const uint64_t per_group = d.mode == MODE_BITMAP ? kBitmapGroupCells : kTableGroupCells;
        d.ngroups = (uint32_t)((total_cells + per_group - 1) / per_group);
        d.max_ovf = d.cap > 0 ? (uint32_t)(maxpts / ((size_t)d.cap + 1) + 1) : 0;
        d.max_list = (uint32_t)maxpts;
        o_store[s] = plan.take((size_t)d.ngroups * 1024);
        o_flag[s] = plan.take((size_t)d.ngroups * sizeof(int4));
        o_acc[s] = plan.take(maxpts * 2 * sizeof(float4));
        o_cl[s] = plan.take(maxpts * sizeof(uint32_t));
        for (int k = 0; k < 3; ++k) o_ovf[s][k] = d.cap > 0 ? plan.take((size_t)d.max_ovf * sizeof(int)) : 0;
        o_ovf[s][3] = d.cap > 0 ? plan.take(maxpts * sizeof(int)) : 0;
        o_ovf[s][4] = d.cap > 0 ? plan.take((size_t)d.max_ovf * kCursorStride * sizeof(int)) : 0;
        o_tot[s] = plan.take(4 * sizeof(int));
    }
    // The rank scan gives a CTA 32 groups of one scale.
    const size_t scan_ctas = (size_t)(h->scale[0].ngroups + 31) / 32 + (size_t)(h->scale[1].ngroups + 31) / 32;
    const size_t o_part = plan.take(scan_ctas * 3 * sizeof(int));
    const size_t o_pbase = plan.take(scan_ctas * 3 * sizeof(int));
    const size_t o_units = plan.take(scan_ctas * sizeof(int));
    const size_t o_vif_start = plan.take(maxpts * sizeof(int));
    const size_t o_vif_cursor = plan.take(maxpts * sizeof(int));
    const size_t o_vif_list = plan.take(maxpts * sizeof(int));
    const size_t o_vif_recs = plan.take(maxpts * sizeof(uint4));
    const size_t o_vif_part = plan.take(((size_t)h->vif_scan_blocks + 1) * sizeof(int));
    const size_t rb_tiles = (maxpts + kTile - 1) / kTile;
    const size_t o_rb_bits = plan.take(maxpts * sizeof(uint32_t));
    const size_t o_rb_counts = plan.take(27 * rb_tiles * sizeof(int));
    const size_t o_rb_base = plan.take((27 * rb_tiles + 27) * sizeof(int));
    h->max_tiles = (c.max_points + kTile - 1) / kTile;
    const size_t tile_ints = (size_t)c.max_batch * h->max_tiles * c.num_experts;
    const size_t o_tc = plan.take(tile_ints * sizeof(int));
    const size_t o_tb = plan.take(tile_ints * sizeof(int));
    const size_t o_status = plan.take(sizeof(int));

    h->slab_bytes = plan.off;
    cudaError_t e = cudaMalloc(&h->slab, h->slab_bytes);
    if (e != cudaSuccess) { h->slab = nullptr; delete h; return EMC2_ERR_CUDA; }
    // The voxel stores must be all-zero between calls; every call restores that.
    e = cudaMemset(h->slab, 0, h->slab_bytes);
    if (e != cudaSuccess) { cudaFree(h->slab); delete h; return EMC2_ERR_CUDA; }
    char* base = static_cast<char*>(h->slab);
    for (int s = 0; s < 2; ++s) {
        ScaleDev& d = h->scale[s];
        d.store = reinterpret_cast<uint32_t*>(base + o_store[s]);
        d.group_info = reinterpret_cast<int4*>(base + o_flag[s]);
        d.acc = reinterpret_cast<float4*>(base + o_acc[s]);
        d.cell_list = reinterpret_cast<uint32_t*>(base + o_cl[s]);
        d.ovf_off = d.cap > 0 ? reinterpret_cast<int*>(base + o_ovf[s][0]) : nullptr;
        d.ovf_vox = d.cap > 0 ? reinterpret_cast<int*>(base + o_ovf[s][1]) : nullptr;
        d.ovf_cell = d.cap > 0 ? reinterpret_cast<uint32_t*>(base + o_ovf[s][2]) : nullptr;
        d.ovf_list = d.cap > 0 ? reinterpret_cast<int*>(base + o_ovf[s][3]) : nullptr;
        d.ovf_cursor = d.cap > 0 ? reinterpret_cast<int*>(base + o_ovf[s][4]) : nullptr;
        d.totals = reinterpret_cast<int*>(base + o_tot[s]);
    }
    h->d_scan_tot = reinterpret_cast<int*>(base + o_part);
    h->d_scan_base = reinterpret_cast<int*>(base + o_pbase);
    h->d_scan_units = reinterpret_cast<int*>(base + o_units);
    h->d_vif_start = reinterpret_cast<int*>(base + o_vif_start);
    h->d_vif_cursor = reinterpret_cast<int*>(base + o_vif_cursor);
    h->d_vif_list = reinterpret_cast<int*>(base + o_vif_list);
    h->d_vif_recs = reinterpret_cast<uint4*>(base + o_vif_recs);
    h->d_vif_part = reinterpret_cast<int*>(base + o_vif_part);
    h->d_rb_bits = reinterpret_cast<uint32_t*>(base + o_rb_bits);
    h->d_rb_counts = reinterpret_cast<int*>(base + o_rb_counts);
    h->d_rb_base = reinterpret_cast<int*>(base + o_rb_base);
    h->d_tile_counts = reinterpret_cast<int*>(base + o_tc);
    h->d_tile_base = reinterpret_cast<int*>(base + o_tb);
    h->d_status = reinterpret_cast<int*>(base + o_status);
    int prio_lo = 0, prio_hi = 0;
    e = cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi);
    if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&h->side, cudaStreamNonBlocking, prio_hi);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_half, cudaEventDisableTiming);
    if (e != cudaSuccess) { emc2_bridge_destroy(h); return EMC2_ERR_CUDA; }
    *out = h;
    return EMC2_OK;
}

static int check_call(emc2_bridge* h, int32_t B, int32_t N) {
    if (!h) return EMC2_ERR_INVALID_ARG;
    if (B < 0 || N < 0 || B > h->cfg.max_batch || N > h->cfg.max_points) return EMC2_ERR_INVALID_ARG;
    return EMC2_OK;
}

static int check_voxelize_args(emc2_bridge* h, int32_t B, int32_t N, const float* d_points,
                               int32_t* const d_coords[2], int32_t* const d_counts[2], float* const d_mean[2],
                               const int32_t capacity[2], const int32_t* d_num_voxels, const float* d_bev) {
    int rc = check_call(h, B, N);
    if (rc != EMC2_OK) return rc;
    const bool empty = B == 0 || N == 0;   // zero-sized buffers may be null
    if ((!d_points && !empty) || !d_coords || !d_counts || !d_mean || !capacity || !d_num_voxels)
        return EMC2_ERR_INVALID_ARG;
    if (!aligned16(d_points) || (d_bev && !aligned16(d_bev))) return EMC2_ERR_INVALID_ARG;
    for (int s = 0; s < 2; ++s) {
        if (!d_coords[s] || !d_counts[s] || !d_mean[s] || capacity[s] < 0) return EMC2_ERR_INVALID_ARG;
        if (!aligned16(d_coords[s])) return EMC2_ERR_INVALID_ARG;
    }
    return EMC2_OK;
}

int emc2_voxelize(emc2_bridge_t* h, int32_t B, int32_t N, const float* d_points,
                  int32_t* const d_coords[2], int32_t* const d_counts[2], float* const d_mean[2],
                  int32_t* const d_point_voxel[2], const int32_t capacity[2], int32_t* d_num_voxels,
                  float* d_bev, void* cuda_stream) {
    int rc = check_voxelize_args(h, B, N, d_points, d_coords, d_counts, d_mean, capacity, d_num_voxels, d_bev);
    if (rc != EMC2_OK) return rc;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return EMC2_ERR_CUDA;
    return launch_voxelize(h, B, N, d_points, d_coords, d_counts, d_mean, d_point_voxel, capacity,
                           d_num_voxels, d_bev, static_cast<cudaStream_t>(cuda_stream));
}

int emc2_project_gather(emc2_bridge_t* h, int32_t B, int32_t N, const float* d_points, const float* d_proj,
                        const float* d_feat, float* d_uvd, uint8_t* d_vis_mask, int8_t* d_cam,
                        float* d_gathered, void* cuda_stream) {
    int rc = check_call(h, B, N);
    if (rc != EMC2_OK) return rc;
    if (B == 0 || N == 0) return EMC2_OK;   // nothing to write
    if (!d_points || !d_proj || !d_feat || !d_uvd || !d_vis_mask || !d_cam || !d_gathered)
        return EMC2_ERR_INVALID_ARG;
    if (!aligned16(d_points) || !aligned16(d_proj) || !aligned16(d_feat) || !aligned16(d_gathered))
        return EMC2_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return EMC2_ERR_CUDA;
    return launch_project_gather(h, B, N, d_points, d_proj, d_feat, d_uvd, d_vis_mask, d_cam, d_gathered,
                                 static_cast<cudaStream_t>(cuda_stream));
}

int emc2_route_dispatch(emc2_bridge_t* h, int32_t B, int32_t N, const float* d_points,
                        const uint8_t* d_vis_mask, const float* d_gathered, uint8_t* d_expert,
                        int32_t* d_offsets, int32_t* d_perm, float* d_points_out, float* d_feat_out,
                        void* cuda_stream) {
    int rc = check_call(h, B, N);
    if (rc != EMC2_OK) return rc;
    if (B == 0) return EMC2_OK;             // nothing to write
    if (!d_offsets) return EMC2_ERR_INVALID_ARG;
    if (N > 0 && (!d_points || !d_vis_mask || !d_gathered || !d_expert || !d_perm || !d_points_out ||
                  !d_feat_out))
        return EMC2_ERR_INVALID_ARG;
    if (!aligned16(d_points) || !aligned16(d_gathered) || !aligned16(d_feat_out)) return EMC2_ERR_INVALID_ARG;
    if (N > 0 && (d_points_out == d_points || d_feat_out == d_gathered)) return EMC2_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return EMC2_ERR_CUDA;
    return launch_route_dispatch(h, B, N, d_points, d_vis_mask, d_gathered, d_expert, d_offsets, d_perm,
                                 d_points_out, d_feat_out, static_cast<cudaStream_t>(cuda_stream));
}

int emc2_bridge_run(emc2_bridge_t* h, int32_t B, int32_t N, const float* d_points, const float* d_proj,
                    const float* d_feat, int32_t* const d_coords[2], int32_t* const d_counts[2],
                    float* const d_mean[2], int32_t* const d_point_voxel[2], const int32_t capacity[2],
                    int32_t* d_num_voxels, float* d_bev, float* d_uvd, uint8_t* d_vis_mask, int8_t* d_cam,
                    float* d_gathered, uint8_t* d_expert, int32_t* d_offsets, int32_t* d_perm,
                    float* d_points_out, float* d_feat_out, void* cuda_stream) {
    // The stage calls validate before they enqueue anything; a host-detected error in stage 2 or
    // 3 - 4 leaves stage 1 enqueued, exactly as three separate calls would.
    if (!h) return EMC2_ERR_INVALID_ARG;
    int rc = check_voxelize_args(h, B, N, d_points, d_coords, d_counts, d_mean, capacity, d_num_voxels, d_bev);
    if (rc != EMC2_OK) return rc;
    // The checks of emc2_project_gather and emc2_route_dispatch.
    int rc2 = EMC2_OK;
    if (B > 0) {
        if (!d_offsets) rc2 = EMC2_ERR_INVALID_ARG;
        else if (N > 0 && (!d_points || !d_proj || !d_feat || !d_uvd || !d_vis_mask || !d_cam ||
                           !d_expert || !d_perm || !d_points_out || !d_feat_out))   // d_gathered may be null
            rc2 = EMC2_ERR_INVALID_ARG;
        else if (!aligned16(d_points) || !aligned16(d_proj) || !aligned16(d_feat) || !aligned16(d_gathered) ||
                 !aligned16(d_feat_out))
            rc2 = EMC2_ERR_INVALID_ARG;
        else if (N > 0 && (d_points_out == d_points || d_feat_out == d_gathered))
            rc2 = EMC2_ERR_INVALID_ARG;
    }
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return EMC2_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaStream_t vox_st = h->overlap ? h->side : st;
    cudaError_t e = cudaSuccess;
    // One pass over the points serves the projection, the routing and the voxelizer's marking; the
    // rest of stage 1 then runs on the side stream beside the row traffic of stages 2 - 4.
    const bool fused_mark = rc2 == EMC2_OK && B > 0 && N > 0 && h->tune[EMC2_TUNE_MARK_IN_PROJECTION] != 0;
    // With two or more frames the batch is taken in two halves: the rows of the first half start to
    // move as soon as ITS points are projected, while the second half is projected on the side stream.
    const int half0 = fused_mark && h->overlap && B >= 2 && h->tune[EMC2_TUNE_SPLIT_BATCH] != 0 ? B / 2 : B;
    if (fused_mark)
        rc = launch_project_route(h, 0, half0, N, d_points, d_proj, d_uvd, d_vis_mask, d_cam, d_expert, true, d_bev, B, st);
    if (rc == EMC2_OK && h->overlap) {
        e = cudaEventRecord(h->ev_fork, st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(h->side, h->ev_fork, 0);
        if (e != cudaSuccess) return check_cuda(h, e);
    }
    if (rc == EMC2_OK && half0 < B) {
        rc = launch_project_route(h, half0, B - half0, N, d_points, d_proj, d_uvd, d_vis_mask, d_cam, d_expert, true,
                                  nullptr, 0, h->side);
        if (rc == EMC2_OK) {
            e = cudaEventRecord(h->ev_half, h->side);
            if (e != cudaSuccess) rc = check_cuda(h, e);
        }
    }
    if (rc == EMC2_OK)
        rc = launch_voxelize(h, B, N, d_points, d_coords, d_counts, d_mean, d_point_voxel, capacity, d_num_voxels,
                             d_bev, vox_st, fused_mark);
    if (rc == EMC2_OK && rc2 == EMC2_OK && B > 0) {
        if (!fused_mark)
            rc2 = launch_project_route(h, 0, B, N, d_points, d_proj, d_uvd, d_vis_mask, d_cam, d_expert, false, nullptr, 0, st);
        if (rc2 == EMC2_OK)
            rc2 = launch_scan_gather_scatter(h, 0, half0, N, d_points, d_feat, d_uvd, d_cam, d_gathered, d_expert,
                                             d_offsets, d_perm, d_points_out, d_feat_out, st);
        if (rc2 == EMC2_OK && half0 < B) {
            e = cudaStreamWaitEvent(st, h->ev_half, 0);
            if (e != cudaSuccess) rc2 = check_cuda(h, e);
            else
                rc2 = launch_scan_gather_scatter(h, half0, B - half0, N, d_points, d_feat, d_uvd, d_cam, d_gathered,
                                                 d_expert, d_offsets, d_perm, d_points_out, d_feat_out, st);
        }
    }
    // Join even after an error, so that `cuda_stream` never runs ahead of stage 1.
    if (h->overlap) {
        e = cudaEventRecord(h->ev_join, h->side);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, h->ev_join, 0);
    }
    if (rc != EMC2_OK) return rc;
    if (rc2 != EMC2_OK) return rc2;
    return check_cuda(h, e);
}

int emc2_voxel_image(emc2_bridge_t* h, int32_t B, int32_t N, int32_t capacity, const int32_t* d_point_voxel,
                     const int32_t* d_counts, const int32_t* d_num_voxels, const uint8_t* d_vis_mask,
                     const float* d_gathered, float* d_vox_img, int32_t* d_vox_img_count, void* cuda_stream) {
    int rc = check_call(h, B, N);
    if (rc != EMC2_OK) return rc;
    if (capacity < 0 || !d_num_voxels) return EMC2_ERR_INVALID_ARG;
    if (B == 0 || N == 0 || capacity == 0) return EMC2_OK;
    if (!d_point_voxel || !d_counts || !d_vis_mask || !d_gathered || !d_vox_img || !d_vox_img_count)
        return EMC2_ERR_INVALID_ARG;
    if (!aligned16(d_gathered) || !aligned16(d_vox_img)) return EMC2_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return EMC2_ERR_CUDA;
    return launch_voxel_image(h, B, N, capacity, d_point_voxel, d_counts, d_num_voxels, d_vis_mask, d_gathered,
                              nullptr, nullptr, nullptr, d_vox_img, d_vox_img_count,
                              static_cast<cudaStream_t>(cuda_stream));
}

int emc2_voxel_image_sampled(emc2_bridge_t* h, int32_t B, int32_t N, int32_t capacity, const int32_t* d_point_voxel,
                             const int32_t* d_counts, const int32_t* d_num_voxels, const float* d_uvd,
                             const int8_t* d_cam, const float* d_feat, float* d_vox_img, int32_t* d_vox_img_count,
                             void* cuda_stream) {
    int rc = check_call(h, B, N);
    if (rc != EMC2_OK) return rc;
    if (capacity < 0 || !d_num_voxels) return EMC2_ERR_INVALID_ARG;
    if (B == 0 || N == 0 || capacity == 0) return EMC2_OK;
    if (!d_point_voxel || !d_counts || !d_uvd || !d_cam || !d_feat || !d_vox_img || !d_vox_img_count)
        return EMC2_ERR_INVALID_ARG;
    if (!aligned16(d_feat) || !aligned16(d_vox_img)) return EMC2_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return EMC2_ERR_CUDA;
    return launch_voxel_image(h, B, N, capacity, d_point_voxel, d_counts, d_num_voxels, nullptr, nullptr, d_uvd,
                              d_cam, d_feat, d_vox_img, d_vox_img_count, static_cast<cudaStream_t>(cuda_stream));
}

int emc2_voxel_image_pooled(emc2_bridge_t* h, int32_t B, int32_t N, int32_t capacity, const int32_t* d_point_voxel,
                            const int32_t* d_counts, const int32_t* d_num_voxels, const float* d_uvd,
                            const int8_t* d_cam, const float* d_feat, int32_t p, float* d_vox_img,
                            int32_t* d_vox_img_count, void* cuda_stream) {
    int rc = check_call(h, B, N);
    if (rc != EMC2_OK) return rc;
    if (capacity < 0 || !d_num_voxels || !is_pow2(p)) return EMC2_ERR_INVALID_ARG;
    if (B == 0 || N == 0 || capacity == 0) return EMC2_OK;
    if (!d_point_voxel || !d_counts || !d_uvd || !d_cam || !d_feat || !d_vox_img || !d_vox_img_count)
        return EMC2_ERR_INVALID_ARG;
    if (!aligned16(d_feat) || !aligned16(d_vox_img)) return EMC2_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return EMC2_ERR_CUDA;
    return launch_voxel_image(h, B, N, capacity, d_point_voxel, d_counts, d_num_voxels, nullptr, nullptr, d_uvd,
                              d_cam, d_feat, d_vox_img, d_vox_img_count, static_cast<cudaStream_t>(cuda_stream), p);
}

int emc2_rulebook(emc2_bridge_t* h, int32_t scale, int32_t capacity, const int32_t* d_coords,
                  const int32_t* d_num_voxels, int32_t* d_rule_offsets, int32_t* d_rule_in, int32_t* d_rule_out,
                  int64_t pair_capacity, void* cuda_stream) {
    if (!h || scale < 0 || scale > 1 || capacity < 0 || pair_capacity < 0) return EMC2_ERR_INVALID_ARG;
    if ((int64_t)capacity > (int64_t)h->cfg.max_batch * h->cfg.max_points) return EMC2_ERR_INVALID_ARG;
    if (!d_num_voxels || !d_rule_offsets) return EMC2_ERR_INVALID_ARG;
    if (capacity > 0 && (!d_coords || !aligned16(d_coords))) return EMC2_ERR_INVALID_ARG;
    if (pair_capacity > 0 && (!d_rule_in || !d_rule_out)) return EMC2_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return EMC2_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (capacity == 0) return check_cuda(h, cudaMemsetAsync(d_rule_offsets, 0, 28 * sizeof(int32_t), st));
    return launch_rulebook(h, scale, capacity, d_coords, d_num_voxels, d_rule_offsets, d_rule_in, d_rule_out,
                           pair_capacity, st);
}

int emc2_occlusion(emc2_bridge_t* h, int32_t B, int32_t N, const float* d_points, const float* d_proj,
                   const uint8_t* d_vis_mask, int32_t cell, float margin, float* d_zbuf, uint8_t* d_occ_mask,
                   uint8_t* d_clear_mask, void* cuda_stream) {
    int rc = check_call(h, B, N);
    if (rc != EMC2_OK) return rc;
    if (!is_pow2(cell) || !(margin >= 0.0f) || !std::isfinite(margin)) return EMC2_ERR_INVALID_ARG;
    if (B == 0) return EMC2_OK;
    if (!d_zbuf || !d_proj || !aligned16(d_proj)) return EMC2_ERR_INVALID_ARG;
    if (N > 0 && (!d_points || !d_vis_mask || !d_occ_mask || !d_clear_mask)) return EMC2_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return EMC2_ERR_CUDA;
    return launch_occlusion(h, B, N, d_points, d_proj, d_vis_mask, cell, margin, reinterpret_cast<uint32_t*>(d_zbuf),
                            d_occ_mask, d_clear_mask, static_cast<cudaStream_t>(cuda_stream));
}

int emc2_bridge_run_host(emc2_bridge_t* h, int32_t B, int32_t N, const float* h_points, const float* h_proj,
                         const float* h_feat, float* d_points, float* d_proj, float* d_feat,
                         int32_t* const d_coords[2], int32_t* const d_counts[2], float* const d_mean[2],
                         int32_t* const d_point_voxel[2], const int32_t capacity[2], int32_t* d_num_voxels,
                         float* d_bev, float* d_uvd, uint8_t* d_vis_mask, int8_t* d_cam, float* d_gathered,
                         uint8_t* d_expert, int32_t* d_offsets, int32_t* d_perm, float* d_points_out,
                         float* d_feat_out, int32_t* h_offsets, int32_t* h_num_voxels, void* cuda_stream) {
    int rc = check_call(h, B, N);
    if (rc != EMC2_OK) return rc;
    const emc2_config_t& c = h->cfg;
    if (B > 0 && (!h_proj || !h_feat || !d_proj || !d_feat || (N > 0 && (!h_points || !d_points))))
        return EMC2_ERR_INVALID_ARG;
    DeviceGuard guard(c.device);
    if (!guard.ok) return EMC2_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaSuccess;
    if (B > 0) {
        const size_t pts = (size_t)B * N * c.point_floats * sizeof(float);
        const size_t prj = (size_t)B * c.num_cameras * 12 * sizeof(float);
        const size_t fts = (size_t)B * c.num_cameras * c.feat_h * c.feat_w * c.feat_c * sizeof(float);
        if (pts) e = cudaMemcpyAsync(d_points, h_points, pts, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(d_proj, h_proj, prj, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(d_feat, h_feat, fts, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return check_cuda(h, e);
    }
    rc = emc2_bridge_run(h, B, N, d_points, d_proj, d_feat, d_coords, d_counts, d_mean, d_point_voxel, capacity,
                         d_num_voxels, d_bev, d_uvd, d_vis_mask, d_cam, d_gathered, d_expert, d_offsets, d_perm,
                         d_points_out, d_feat_out, cuda_stream);
    if (rc != EMC2_OK) return rc;
    if (h_offsets && d_offsets && B > 0)
        e = cudaMemcpyAsync(h_offsets, d_offsets, (size_t)B * (c.num_experts + 1) * sizeof(int32_t),
                            cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && h_num_voxels && d_num_voxels)
        e = cudaMemcpyAsync(h_num_voxels, d_num_voxels, 2 * sizeof(int32_t), cudaMemcpyDeviceToHost, st);
    return check_cuda(h, e);
}

int emc2_features_channels_last(emc2_bridge_t* h, int32_t B, const float* d_planar, float* d_feat,
                                void* cuda_stream) {
    if (!h || B < 0 || B > h->cfg.max_batch) return EMC2_ERR_INVALID_ARG;
    if (B == 0) return EMC2_OK;
    if (!d_planar || !d_feat || !aligned16(d_planar) || !aligned16(d_feat) || d_planar == d_feat)
        return EMC2_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return EMC2_ERR_CUDA;
    return launch_channels_last(h, B, d_planar, d_feat, static_cast<cudaStream_t>(cuda_stream));
}

int emc2_pool_features(emc2_bridge_t* h, int32_t B, int32_t p, const float* d_feat, float* d_pooled,
                       void* cuda_stream) {
    if (!h || B < 0 || B > h->cfg.max_batch || p < 1) return EMC2_ERR_INVALID_ARG;
    if (B == 0) return EMC2_OK;
    if (!d_feat || !d_pooled || !aligned16(d_feat) || !aligned16(d_pooled) || d_feat == d_pooled)
        return EMC2_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return EMC2_ERR_CUDA;
    return launch_pool_features(h, B, p, d_feat, d_pooled, static_cast<cudaStream_t>(cuda_stream));
}

int emc2_scene_route(emc2_bridge_t* h, int32_t B, const int32_t* d_offsets, const uint8_t* priority,
                     int32_t min_points, int32_t* d_scene_expert, void* cuda_stream) {
    if (!h || B < 0 || B > h->cfg.max_batch || !priority) return EMC2_ERR_INVALID_ARG;
    if (B == 0) return EMC2_OK;
    if (!d_offsets || !d_scene_expert) return EMC2_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return EMC2_ERR_CUDA;
    return launch_scene_route(h, B, d_offsets, priority, min_points, d_scene_expert,
                              static_cast<cudaStream_t>(cuda_stream));
}

int emc2_bridge_set_overlap(emc2_bridge_t* h, int enable) {
    if (!h) return EMC2_ERR_INVALID_ARG;
    h->overlap = enable != 0;
    return EMC2_OK;
}

int emc2_bridge_set_tuning(emc2_bridge_t* h, int32_t knob, int32_t value) {
    if (!h || knob < 0 || knob >= EMC2_TUNE_KNOBS) return EMC2_ERR_INVALID_ARG;
    static const int kMaxValue[EMC2_TUNE_KNOBS] = {3, 1, 2, 2, 1};
    if (value < 0 || value > kMaxValue[knob]) return EMC2_ERR_INVALID_ARG;
    if (knob == EMC2_TUNE_DEDUP_FINE || knob == EMC2_TUNE_DEDUP_PILLARS) {
        const int s = knob == EMC2_TUNE_DEDUP_FINE ? 0 : 1;
        if (value != 0) {                         // the other designs bring scratch of their own
            DeviceGuard guard(h->cfg.device);
            if (!guard.ok) return EMC2_ERR_CUDA;
            const int rc = dedup_arm_alloc(h);
            if (rc != EMC2_OK) return rc;
        }
        h->scale[s].design = value;
        h->scale[s].point_rank = value ? h->arm.point_rank[s] : nullptr;
    }
    h->tune[knob] = value;
    return EMC2_OK;
}

int emc2_bridge_status(emc2_bridge_t* h, void* cuda_stream) {
    if (!h) return EMC2_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return EMC2_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, h->d_status, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->d_status, 0, sizeof(int), st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return check_cuda(h, e);
    if (word & 2) return EMC2_ERR_TIMEOUT;
    if (word & 1) return EMC2_ERR_CAPACITY;
    if (word & 4) return EMC2_ERR_INVALID_ARG;
    if (word & 8) return EMC2_ERR_INTERNAL;
    return EMC2_OK;
}

int emc2_bridge_destroy(emc2_bridge_t* h) {
    if (!h) return EMC2_OK;
    DeviceGuard guard(h->cfg.device);
    int rc = EMC2_OK;
    for (ProfRec& r : h->recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    for (cudaEvent_t e : h->event_pool) cudaEventDestroy(e);
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->ev_join) cudaEventDestroy(h->ev_join);
    if (h->ev_half) cudaEventDestroy(h->ev_half);
    if (h->side) cudaStreamDestroy(h->side);
    if (h->slab && cudaFree(h->slab) != cudaSuccess) rc = EMC2_ERR_CUDA;
    if (h->arm.slab && cudaFree(h->arm.slab) != cudaSuccess) rc = EMC2_ERR_CUDA;
    delete h;
    return rc;
}

const char* emc2_status_string(int status) {
    switch (status) {
        case EMC2_OK: return "ok";
        case EMC2_ERR_INVALID_ARG: return "invalid argument";
        case EMC2_ERR_BAD_CONFIG: return "bad configuration";
        case EMC2_ERR_CUDA: return "CUDA runtime error";
        case EMC2_ERR_CAPACITY: return "more unique voxels than capacity";
        case EMC2_ERR_TIMEOUT: return "bounded device wait timed out";
        case EMC2_ERR_INTERNAL: return "internal error";
        case EMC2_ERR_TOO_LARGE: return "call exceeds the fixed scratch area";
        default: return "unknown status";
    }
}

int emc2_bridge_last_cuda_error(const emc2_bridge_t* h) { return h ? h->last_cuda_error : 0; }
size_t emc2_bridge_scratch_bytes(const emc2_bridge_t* h) { return h ? h->slab_bytes + h->arm.bytes : 0; }

int emc2_bridge_kernel_kinds(void) { return K_KINDS; }
const char* emc2_bridge_kernel_name(int kind) { return kind >= 0 && kind < K_KINDS ? kKernelNames[kind] : ""; }

int emc2_bridge_profile_enable(emc2_bridge_t* h, int enable) {
    if (!h) return EMC2_ERR_INVALID_ARG;
    h->profiling = enable != 0;
    return EMC2_OK;
}

int emc2_bridge_profile_read(emc2_bridge_t* h, int64_t* launches, double* ms, int reset) {
    if (!h) return EMC2_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    int rc = EMC2_OK;
    for (ProfRec& r : h->recs) {
        float t = 0.f;
        cudaError_t e = cudaEventSynchronize(r.b);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&t, r.a, r.b);
        if (e == cudaSuccess) h->ms[r.kind] += t; else rc = check_cuda(h, e);
        h->event_pool.push_back(r.a);
        h->event_pool.push_back(r.b);
    }
    h->recs.clear();
    for (int k = 0; k < K_KINDS; ++k) {
        if (launches) launches[k] = h->launches[k];
        if (ms) ms[k] = h->ms[k];
        if (reset) { h->launches[k] = 0; h->ms[k] = 0.0; }
    }
    return rc;
}

int emc2_bridge_profile_timeline(emc2_bridge_t* h, int32_t* kinds, float* start_ms, float* end_ms,
                                 int32_t capacity) {
    if (!h || capacity < 0 || (capacity > 0 && (!kinds || !start_ms || !end_ms))) return EMC2_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    int n = 0, rc = EMC2_OK;
    cudaEvent_t origin = h->recs.empty() ? nullptr : h->recs.front().a;
    for (ProfRec& r : h->recs) {
        float t0 = 0.f, t1 = 0.f;
        cudaError_t e = cudaEventSynchronize(r.b);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&t0, origin, r.a);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&t1, origin, r.b);
        if (e != cudaSuccess) rc = check_cuda(h, e);
        else if (n < capacity) { kinds[n] = r.kind; start_ms[n] = t0; end_ms[n] = t1; ++n; }
    }
    for (ProfRec& r : h->recs) { h->event_pool.push_back(r.a); h->event_pool.push_back(r.b); }
    h->recs.clear();
    return rc != EMC2_OK ? rc : n;
}

}  // extern "C"
