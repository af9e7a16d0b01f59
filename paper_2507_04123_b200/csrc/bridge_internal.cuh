// Internal declarations shared by the bridge's translation units (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "emc2_bridge.h"

namespace emc2 {

constexpr int kTile = 256;           // points per CTA tile in the per-point kernels
constexpr int kThreads = 256;
constexpr int kBitmapGroupCells = 32 * 4 * 32;  // a 1 KB bitmap group: 32 sectors of four {bits, rank} pairs
constexpr int kTableGroupCells = 32 * 2;         // a 1 KB table group: 32 sectors of two cell records
constexpr int kMaxTableCells = 1 << 24;  // per-cell records up to 16 Mi cells per batch (256 MB)
constexpr int kCursorStride = 8;         // ints between list cursors: one 32-byte sector each

// Kernel kinds, for the launch counters and the optional event timing.
enum KernelKind {
    K_VOX_MARK = 0,
    K_VOX_COUNT,
    K_VOX_PREFIX,
    K_VOX_RANK,
    K_VOX_ACCUM,
    K_VOX_OVER_FIND,
    K_VOX_OVER_FILL,
    K_VOX_FINALIZE,
    K_ARM_KEYS,
    K_ARM_SORT,
    K_ARM_HASH,
    K_ARM_RANK,
    K_PROJECT_GATHER,
    K_PROJECT_ROUTE,
    K_GATHER_SCATTER,
    K_ROUTE_HIST,
    K_ROUTE_SCAN,
    K_DISPATCH_SCATTER,
    K_SCENE_ROUTE,
    K_POOL_FEATURES,
    K_VIF_SCAN,
    K_VIF_FILL,
    K_VIF_MEAN,
    K_VIF_SAMPLE,
    K_OCCL_FILL,
    K_OCCL_SPLAT,
    K_OCCL_TEST,
    K_CHANNELS_LAST,
    K_RB_MARK,
    K_RB_COUNT,
    K_RB_SCAN,
    K_RB_FILL,
    K_RB_CLEAR,
    K_KINDS
};

enum ScaleMode { MODE_BITMAP = 0, MODE_TABLE = 1 };

// Division of any 32-bit unsigned number by a fixed divisor with a multiply and two shifts
// (Granlund and Montgomery, "Division by invariant integers using multiplication", 1994).
struct FastDiv {
    uint32_t d, m, s1, s2;
#ifdef __CUDACC__
    __device__ __forceinline__ void divmod(uint32_t n, uint32_t& q, uint32_t& r) const {
        const uint32_t t = __umulhi(m, n);
        const uint32_t qq = (t + ((n - t) >> s1)) >> s2;
        r = n - qq * d;
        q = qq;
    }
#endif
};

inline FastDiv make_fast_div(uint32_t d) {
    FastDiv f;
    uint32_t L = 0;
    while (L < 32 && ((uint64_t)1 << L) < d) ++L;
    f.d = d;
    f.m = (uint32_t)((((uint64_t)1 << 32) * (((uint64_t)1 << L) - d)) / d + 1);
    f.s1 = L < 1 ? L : 1;
    f.s2 = L > 0 ? L - 1 : 0;
    return f;
}

// Per-scale grid description and scratch pointers, passed to kernels by value.
struct ScaleDev {
    float mn[3];
    float vs[3];
    int dims[3];            // Gx, Gy, Gz
    FastDiv div[3];         // division by Gx, Gy, Gz
    int cap;                // 0 = none
    int mode;               // ScaleMode
    uint32_t cells;         // cells per frame
    uint32_t ngroups;       // 1 KB groups of `store` for the largest batch
    uint32_t max_ovf;       // most cells that can exceed the cap
    uint32_t max_list;      // entries of acc / cell_list / ovf_list: the most points of a call
    uint32_t* store;        // bitmap: {bits, rank} per 32 cells; table: {count, rank, over-cap rank, -} per cell;
                            // bits / counts are zero between calls
    int4* group_info;       // [ngroups] {voxels, cells over the cap, their points} of the group (rewritten by
                            // every call)
    float4* acc;            // [max voxels][2] per-voxel accumulators
    uint32_t* cell_list;    // [max voxels] cell id of each unique voxel (table stores: bit 31 = over the cap)
    int* ovf_off;           // per cell over the cap j: start of its points in ovf_list
    int* ovf_cursor;        // per cell over the cap j: points appended so far, at [j * kCursorStride]
    uint32_t* ovf_cell;     // per cell over the cap j: its cell id
    int* ovf_vox;           // per cell over the cap j: its row m in the unique list
    int* ovf_list;          // global point indices of the points in cells over the cap
    int design;             // dedup design of this scale: 0 = this direct-addressed store, 1 = hash, 2 = sort
                            // (dedup_arms.cu); with 1 or 2 the store is not used and rows come from point_rank
    const int* point_rank;  // design != 0: [points of the call] row of every point's voxel, -1 if outside
    int* totals;            // [0] voxels, [1] cells over the cap, [2] points in cells over the cap, [3] CTAs of the rank scan that found voxels
};

// Routing tables as the kernels take them (Sec. 3.2 distance rule, per point with visibility).
struct RouteParams {
    int T, E;
    float thr2[EMC2_MAX_THRESHOLDS];    // squared thresholds
    uint8_t lut[16];                    // [visible ? 8 : 0] + number of thresholds reached -> expert
};

// Scratch of the alternative dedup designs (allocated when one is first selected).
struct DedupArm {
    void* slab = nullptr;
    size_t bytes = 0;
    uint32_t* keys[2] = {nullptr, nullptr};     // sort buffers (ping-pong): cell ids ...
    uint32_t* vals[2] = {nullptr, nullptr};     // ... and point indices (hash design: the unique ids)
    int* counts = nullptr;                      // [256][tiles] digit counts of a radix pass
    int* row_tot = nullptr;                     // [256] totals per digit
    int* tile_tot = nullptr;                    // run heads per tile
    int* point_rank[2] = {nullptr, nullptr};    // per scale
    uint32_t* tab_keys = nullptr;               // hash table: cell ids ...
    int* tab_rows = nullptr;                    // ... and their rows
    int* d_total = nullptr;
    uint32_t slots = 0;
};

struct ProfRec {
    int kind;
    cudaEvent_t a, b;
};

}  // namespace emc2

struct emc2_bridge {
    emc2_config_t cfg;
    emc2::ScaleDev scale[2];
    float thr2[EMC2_MAX_THRESHOLDS];
    void* slab = nullptr;
    size_t slab_bytes = 0;
    int* d_status = nullptr;       // sticky device status word
    int* d_tile_counts = nullptr;  // [B, tiles per frame, E]
    int* d_tile_base = nullptr;    // same shape, exclusive bases
    int* d_scan_tot = nullptr;     // [CTAs of the voxel rank scan, both scales][3] per-CTA totals
    int* d_scan_base = nullptr;    // same shape: their exclusive prefix sums inside each scale
    int* d_scan_units = nullptr;   // per scale the CTAs that found voxels
    int* d_vif_start = nullptr;    // emc2_voxel_image: [max points] list starts, cursors, lists
    int* d_vif_cursor = nullptr;
    int* d_vif_list = nullptr;
    uint4* d_vif_recs = nullptr;   // emc2_voxel_image_sampled: [max points] tap records in list order
    int* d_vif_part = nullptr;     // [vif_scan_blocks]
    int vif_scan_blocks = 0;
    uint32_t* d_rb_bits = nullptr;  // emc2_rulebook: [max points] neighbour bits per voxel
    int* d_rb_counts = nullptr;    // [27][voxel tiles] pairs per (offset, tile), and their prefix sums
    int* d_rb_base = nullptr;
    int max_tiles = 0;
    int tune[EMC2_TUNE_KNOBS] = {0, 1, 0, 0, 0};   // emc2_bridge_set_tuning
    emc2::DedupArm arm;
    int num_sms = 0;               // multiprocessors of the handle's device
    bool overlap = true;           // emc2_bridge_run puts stage 1 on `side`
    cudaStream_t side = nullptr;   // stream of stage 1 inside emc2_bridge_run
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr, ev_half = nullptr;
    int last_cuda_error = 0;
    bool profiling = false;
    int64_t launches[emc2::K_KINDS] = {0};
    double ms[emc2::K_KINDS] = {0};
    std::vector<emc2::ProfRec> recs;
    std::vector<cudaEvent_t> event_pool;
};

namespace emc2 {

// Brackets a launch with events when profiling; always counts it.
struct LaunchScope {
    emc2_bridge* h;
    int kind;
    cudaStream_t st;
    cudaEvent_t a = nullptr, b = nullptr;
    LaunchScope(emc2_bridge* h_, int kind_, cudaStream_t st_);
    ~LaunchScope();
};

int check_cuda(emc2_bridge* h, cudaError_t e);

// `marked`: the cells of this batch are already marked and the BEV image zeroed (by the projection
// kernel of the one-call path); the marking pass is then skipped.
int launch_voxelize(emc2_bridge* h, int B, int N, const float* d_points, int32_t* const d_coords[2],
                    int32_t* const d_counts[2], float* const d_mean[2], int32_t* const d_point_voxel[2],
                    const int32_t capacity[2], int32_t* d_num_voxels, float* d_bev, cudaStream_t st,
                    bool marked = false);
int dedup_arm_alloc(emc2_bridge* h);
int launch_dedup_arm(emc2_bridge* h, int s, int design, int B, int N, const float* d_points, int capacity,
                     int32_t* d_num_voxels, cudaStream_t st);
int launch_project_gather(emc2_bridge* h, int B, int N, const float* d_points, const float* d_proj,
                          const float* d_feat, float* d_uvd, uint8_t* d_vis_mask, int8_t* d_cam,
                          float* d_gathered, cudaStream_t st);
int launch_route_dispatch(emc2_bridge* h, int B, int N, const float* d_points, const uint8_t* d_vis_mask,
                          const float* d_gathered, uint8_t* d_expert, int32_t* d_offsets, int32_t* d_perm,
                          float* d_points_out, float* d_feat_out, cudaStream_t st);

inline RouteParams route_params(const emc2_bridge* h) {
    RouteParams rp;
    rp.T = h->cfg.num_thresholds;
    rp.E = h->cfg.num_experts;
    for (int k = 0; k < EMC2_MAX_THRESHOLDS; ++k) rp.thr2[k] = h->thr2[k];
    for (int k = 0; k < 16; ++k) rp.lut[k] = h->cfg.lut[k >> 3][k & 7];
    return rp;
}

int launch_occlusion(emc2_bridge* h, int B, int N, const float* d_points, const float* d_proj,
                     const uint8_t* d_vis_mask, int cell, float margin, uint32_t* d_zbuf, uint8_t* d_occ_mask,
                     uint8_t* d_clear_mask, cudaStream_t st);
int voxel_image_scan_max_blocks();
int launch_voxel_image(emc2_bridge* h, int B, int N, int capacity, const int32_t* d_point_voxel,
                       const int32_t* d_counts, const int32_t* d_num_voxels, const uint8_t* d_vis_mask,
                       const float* d_gathered, const float* d_uvd, const int8_t* d_cam, const float* d_feat,
                       float* d_vox_img, int32_t* d_vox_img_count, cudaStream_t st, int pool = 1);
int launch_rulebook(emc2_bridge* h, int scale, int capacity, const int32_t* d_coords, const int32_t* d_num_voxels,
                    int32_t* d_rule_offsets, int32_t* d_rule_in, int32_t* d_rule_out, long long pair_capacity,
                    cudaStream_t st);
int launch_channels_last(emc2_bridge* h, int B, const float* d_planar, float* d_feat, cudaStream_t st);
int launch_pool_features(emc2_bridge* h, int B, int p, const float* d_feat, float* d_pooled, cudaStream_t st);
int launch_scene_route(emc2_bridge* h, int B, const int32_t* d_offsets, const uint8_t* priority, int min_points,
                       int32_t* d_scene_expert, cudaStream_t st);
// Tile histograms (handle scratch) of frames [b0, b0 + B) -> d_offsets (of frame b0 on) and tile bases.
void launch_route_scan(emc2_bridge* h, int b0, int B, int tiles, int N, int32_t* d_offsets, cudaStream_t st);
// Stages 2 - 4 in one pass over the feature rows (the one-call path), in two parts: projection +
// routing per point (which, with `d_bev_to_zero`/`mark`, also marks the voxel cells of both scales
// and zeroes the BEV image, so that stage 1 reads the points once less), then offsets + rows.
int launch_project_route(emc2_bridge* h, int b0, int B, int N, const float* d_points, const float* d_proj,
                         float* d_uvd, uint8_t* d_vis_mask, int8_t* d_cam, uint8_t* d_expert, bool mark,
                         float* d_bev_to_zero, int bev_frames, cudaStream_t st);
int launch_scan_gather_scatter(emc2_bridge* h, int b0, int B, int N, const float* d_points, const float* d_feat,
                               const float* d_uvd, const int8_t* d_cam, float* d_gathered, const uint8_t* d_expert,
                               int32_t* d_offsets, int32_t* d_perm, float* d_points_out, float* d_feat_out,
                               cudaStream_t st);

// ---------------------------------------------------------------- device helpers
#ifdef __CUDACC__

// Loads `nfloats` consecutive floats starting at a 16-byte aligned address into shared
// memory with 128-bit loads (scalar loads for a ragged tail).
__device__ __forceinline__ void load_tile_f32(const float* __restrict__ src, int nfloats, float* smem) {
    const int nvec = nfloats >> 2;
    const float4* s4 = reinterpret_cast<const float4*>(src);
    float4* d4 = reinterpret_cast<float4*>(smem);
    for (int i = threadIdx.x; i < nvec; i += blockDim.x) d4[i] = __ldg(s4 + i);
    for (int i = (nvec << 2) + threadIdx.x; i < nfloats; i += blockDim.x) smem[i] = __ldg(src + i);
}

// Cell index along one axis: one fp32 subtract, one IEEE fp32 divide, floor.  -1 if outside.
__device__ __forceinline__ int axis_cell(float p, float mn, float vs, int dim) {
    float q = __fdiv_rn(__fsub_rn(p, mn), vs);
    float f = floorf(q);
    // NaN fails both comparisons; +-inf fails one of them.
    if (!(f >= 0.0f) || !(f < (float)dim)) return -1;
    return (int)f;
}

// Cell id of a point inside the whole batch, or 0xFFFFFFFF if outside the grid.
__device__ __forceinline__ uint32_t cell_of(const ScaleDev& g, float x, float y, float z, int b) {
    int ix = axis_cell(x, g.mn[0], g.vs[0], g.dims[0]);
    int iy = axis_cell(y, g.mn[1], g.vs[1], g.dims[1]);
    int iz = axis_cell(z, g.mn[2], g.vs[2], g.dims[2]);
    if ((ix | iy | iz) < 0) return 0xFFFFFFFFu;
    return (((uint32_t)b * g.dims[2] + iz) * g.dims[1] + iy) * g.dims[0] + ix;
}

// Marks the cells of one point in both scales' stores: one fire-and-forget reduction each (OR into
// the bit word, ADD into the cell's point count).
__device__ __forceinline__ void mark_point(const ScaleDev& s0, const ScaleDev& s1, float x, float y, float z, int b) {
#pragma unroll
    for (int sc = 0; sc < 2; ++sc) {
        const ScaleDev& g = sc ? s1 : s0;
        if (g.design) continue;                   // another dedup design: no store to mark
        const uint32_t cell = cell_of(g, x, y, z, b);
        if (cell == 0xFFFFFFFFu) continue;
        // Results unused: these compile to reductions, which the thread does not wait for.
        if (g.mode == MODE_BITMAP) atomicOr(&g.store[2 * (size_t)(cell >> 5)], 1u << (cell & 31u));
        else atomicAdd(&g.store[4 * (size_t)cell], 1u);
    }
}

__device__ __forceinline__ int warp_sum(int v) { return __reduce_add_sync(0xFFFFFFFFu, v); }

// ---- bilinear sampling of the channels-last feature maps (used by every kernel that blends rows)
constexpr uint32_t kZeroRow = 0xFFFFFFFFu;

__device__ __forceinline__ float4 blend(const float4& f00, const float4& f01, const float4& f10, const float4& f11,
                                        float wx, float wy) {
    const float ax = 1.0f - wx, ay = 1.0f - wy;
    float4 o;
    o.x = ay * (ax * f00.x + wx * f01.x) + wy * (ax * f10.x + wx * f11.x);
    o.y = ay * (ax * f00.y + wx * f01.y) + wy * (ax * f10.y + wx * f11.y);
    o.z = ay * (ax * f00.z + wx * f01.z) + wy * (ax * f10.z + wx * f11.z);
    o.w = ay * (ax * f00.w + wx * f01.w) + wy * (ax * f10.w + wx * f11.w);
    return o;
}

// Tap record of a point seen by camera `cam` of frame b at pixel (u, v): {float4 index of tap
// (y0, x0), clamp flags, wx, wy}; kZeroRow in .x for a point no camera sees.
__device__ __forceinline__ uint4 tap_record(int b, int cam, float u, float v, int K, int Hf, int Wf, int cf4,
                                            float inv_stride, float offset) {
    uint4 rec = make_uint4(kZeroRow, 0u, 0u, 0u);
    if (cam >= 0 && cam < K) {
        // Texel coordinates: one fp32 subtraction, then an exact scaling (the stride is a power of
        // two).  Taps are clamped to the map on every side.
        const float fx = __fsub_rn(u, offset) * inv_stride, fy = __fsub_rn(v, offset) * inv_stride;
        const float flx = floorf(fx), fly = floorf(fy);
        int x0 = (int)flx, y0 = (int)fly;
        const int x1 = max(min(x0 + 1, Wf - 1), 0), y1 = max(min(y0 + 1, Hf - 1), 0);
        x0 = max(min(x0, Wf - 1), 0);
        y0 = max(min(y0, Hf - 1), 0);
        const uint32_t map = ((uint32_t)b * K + cam) * Hf;
        rec.x = ((map + y0) * Wf + x0) * (uint32_t)cf4;
        rec.y = (uint32_t)(x1 - x0) | ((uint32_t)(y1 - y0) << 1);
        rec.z = __float_as_uint(fx - flx);
        rec.w = __float_as_uint(fy - fly);
    }
    return rec;
}

// Blended feature column c of the row described by `rec` (zeros for kZeroRow).
__device__ __forceinline__ float4 gather_column(const float4* __restrict__ feat, const uint4& rec, int c, uint32_t cf4,
                                                uint32_t row_stride) {
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    if (rec.x != kZeroRow) {
        const float4* p = feat + rec.x + c;
        const uint32_t dx = (rec.y & 1u) ? cf4 : 0u, dy = (rec.y & 2u) ? row_stride : 0u;
        const float4 f00 = __ldg(p), f01 = __ldg(p + dx), f10 = __ldg(p + dy), f11 = __ldg(p + dy + dx);
        o = blend(f00, f01, f10, f11, __uint_as_float(rec.z), __uint_as_float(rec.w));
    }
    return o;
}


#endif  // __CUDACC__

}  // namespace emc2
