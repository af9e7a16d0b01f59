// Fusion by voxel (Fig. 5): the image features of the pixels that share a voxel's 3-D coordinate
// go with that voxel, voxels without such pixels get zero rows.  The pixels with a 3-D coordinate
// are the projected LiDAR points, so voxel m receives the mean of the gathered rows of its kept
// points that some camera sees.
//
// Rows are 256/320 bytes: adding them up with reductions would cost twenty 16-byte requests per
// point.  Instead the points are listed per voxel and each voxel reads its points' rows whole:
//   vif_scan   cooperative launch: exclusive prefix sum of the voxels' kept-point counts (the
//              prefix-sum indexing of Sec. 3.6) -> start of every voxel's list; cursors cleared.
//   vif_fill   every kept point takes a ticket in its voxel's list (one atomic with return).
//   vif_mean   16 voxels x Cf/4 columns of threads per CTA: a voxel's threads walk its list and
//              read each visible point's row with one contiguous 128-bit load per thread.
//   vif_sample the same, but the rows are blended from the feature maps on the spot
//              (emc2_voxel_image_sampled: no [points, Cf] buffer at all); for it vif_fill stores
//              each listed point's tap record (16 bytes) in place of its index.
#include <cooperative_groups.h>

#include "bridge_internal.cuh"

namespace cg = cooperative_groups;

namespace emc2 {
namespace {

struct VifArgs {
    const int32_t* pv;          // [total] row of the point's voxel, -1 if none
    const int32_t* counts;      // [M] kept points per voxel
    const int32_t* num_voxels;  // device: voxels found by emc2_voxelize for this scale
    const uint8_t* vis;         // [total], or null: a point is visible iff cam[i] >= 0
    const float4* gathered;     // [total, cf4] (vif_mean)
    const int8_t* cam;          // [total] camera of every point (vif_sample)
    const float* uvd;           // [total, 3] pixel and depth in that camera (vif_sample)
    const float4* feat;         // feature maps (vif_sample)
    int N, K, Hf, Wf;
    float inv_stride, offset;
    int pool, Hp, Wp;           // pool > 1: taps are p x p window means of the maps (Multiscale Pooling folded
                                // into the sampling); Hp x Wp is the pooled map, inv_stride / offset describe it
    float4* vox_img;            // [capacity, cf4]
    int32_t* vox_cnt;           // [capacity]
    int* start;                 // [capacity] first list slot of each voxel
    int* cursor;                // [capacity]
    int* list;                  // [total] point indices; bitwise complement for points no camera sees
    uint4* recs;                // [total] vif_sample: tap record of every listed point, in list order
    int* part;                  // [gridDim.x]
    int* bad;                   // set by vif_scan when counts[] add up to more than there are points
    int* status;
    long long total;
    int capacity, cf4;
};

__device__ __forceinline__ int voxels_in_use(const VifArgs& a) { return min(*a.num_voxels, a.capacity); }

// Every thread owns a run of consecutive voxels.  CTA totals, grid barrier, then the prefix.
__global__ void __launch_bounds__(kThreads) vif_scan_kernel(VifArgs a) {
    __shared__ int wsum[kThreads / 32];
    __shared__ int s_base;
    cg::grid_group grid = cg::this_grid();
    const int M = voxels_in_use(a);
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const long long nthreads = (long long)gridDim.x * kThreads;
    const int per = (int)((M + nthreads - 1) / nthreads);
    const long long lo64 = ((long long)blockIdx.x * kThreads + t) * per;
    const int lo = (int)min((long long)M, lo64), hi = (int)min((long long)M, lo64 + per);
    // Sums saturate at one more than the points of the call (at most 2^24 + 1): they cannot wrap, and
    // counts[] that add up to more than the points are still seen as such.
    const int limit = (int)min(a.total, (long long)1 << 24) + 1;
    auto count_of = [&](int m) { return min(max(a.counts[m], 0), limit); };
    int sum = 0;
    for (int m = lo; m < hi; ++m) sum = min(sum + count_of(m), limit);
    int inc = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= d) inc = min(inc + y, limit);
    }
    if (lane == 31) wsum[warp] = inc;
    __syncthreads();
    int before = 0, cta_total = 0;
    for (int w = 0; w < kThreads / 32; ++w) {
        if (w < warp) before = min(before + wsum[w], limit);
        cta_total = min(cta_total + wsum[w], limit);
    }
    if (t == 0) a.part[blockIdx.x] = cta_total;
    grid.sync();
    if (warp == 0) {
        int v = 0;
        for (int c = lane; c < (int)blockIdx.x; c += 32) v = min(v + a.part[c], limit);
        v = min(warp_sum(v), limit);                      // 32 terms of at most 2^24 + 1
        if (lane == 0) s_base = v;
    }
    __syncthreads();
    // counts[] that add up to more than the points of the call are not the voxelizer's counts for this
    // batch: the lists would not fit the list array, so the later kernels do nothing.
    if (blockIdx.x == gridDim.x - 1 && t == 0) {
        const int inconsistent = (long long)s_base + cta_total > a.total ? 1 : 0;
        *a.bad = inconsistent;
        if (inconsistent) atomicOr(a.status, 4);
    }
    int run = min(s_base + before, limit) + inc - sum;      // exact whenever the counts are consistent
    for (int m = lo; m < hi; ++m) {
        a.start[m] = run;
        a.cursor[m] = 0;
        run = min(run + count_of(m), limit);
    }
}

__global__ void __launch_bounds__(kThreads) vif_fill_kernel(VifArgs a) {
    if (*a.bad) return;
    const int M = voxels_in_use(a);
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < a.total; i += (long long)gridDim.x * kThreads) {
        const int m = a.pv[i];
        if (m < 0 || m >= M) continue;
        // What goes into the list first (its loads do not wait for the ticket), then the ticket.
        int entry = 0;
        uint4 rec = make_uint4(kZeroRow, 0u, 0u, 0u);
        if (a.vis) {
            entry = a.vis[i] ? (int)i : ~(int)i;
        } else {                                        // rows will be blended from the maps: keep the taps
            // pooled: the record addresses a TEXEL of the pooled map (not a float4 of a row), see pooled_column
            rec = a.pool > 1 ? tap_record((int)(i / a.N), (int)a.cam[i], a.uvd[3 * i], a.uvd[3 * i + 1], a.K, a.Hp, a.Wp, 1,
                                          a.inv_stride, a.offset)
                             : tap_record((int)(i / a.N), (int)a.cam[i], a.uvd[3 * i], a.uvd[3 * i + 1], a.K, a.Hf, a.Wf,
                                          a.cf4, a.inv_stride, a.offset);
        }
        const int pos = a.start[m] + atomicAdd(&a.cursor[m], 1);
        // Inside the list whenever counts[] are the kept-point counts of pv[] (the voxelizer's outputs
        // for this batch); anything else must not index out of range.
        if ((unsigned)pos >= (unsigned)a.total) continue;
        if (a.vis) a.list[pos] = entry;
        else a.recs[pos] = rec;
    }
}

// CF4 > 0: Cf/4 known at compile time, blockDim.x == 16 * CF4.  CF4 == 0: any Cf, 256 threads.
template <int CF4>
__global__ void __launch_bounds__(CF4 > 0 ? 16 * CF4 : kThreads) vif_mean_kernel(VifArgs a) {
    if (*a.bad) return;
    const int M = voxels_in_use(a);
    const int cf4 = CF4 > 0 ? CF4 : a.cf4;
    const int rows = (int)blockDim.x / cf4;                  // voxels a CTA handles at a time
    const int r = (int)threadIdx.x / cf4, c = (int)threadIdx.x - r * cf4;
    if (r >= rows) return;
    // Two voxels per thread and round: their loads (list start and length, first list entry, first
    // row) do not depend on one another and are in flight together.
    const int stride = gridDim.x * rows;
    for (int m0 = blockIdx.x * rows + r; m0 < M; m0 += 2 * stride) {
        int mm[2] = {m0, m0 + stride}, s0[2], n[2], first[2], seen[2] = {0, 0};
        float4 acc[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const bool ok = mm[u] < M;
            s0[u] = ok ? a.start[mm[u]] : 0;
            n[u] = ok ? min(a.counts[mm[u]], a.cursor[mm[u]]) : 0;   // never past what this call appended
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) first[u] = n[u] > 0 ? a.list[s0[u]] : -1;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (first[u] >= 0) {
                acc[u] = __ldcs(a.gathered + (size_t)first[u] * cf4 + c);
                seen[u] = 1;
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            for (int k = 1; k < n[u]; k += 4) {            // four entries in flight; summed in list order
                int idx[4];
                float4 v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) idx[j] = k + j < n[u] ? a.list[s0[u] + k + j] : -1;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (idx[j] >= 0) v[j] = __ldcs(a.gathered + (size_t)idx[j] * cf4 + c);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (idx[j] < 0) continue;
                    acc[u].x += v[j].x; acc[u].y += v[j].y; acc[u].z += v[j].z; acc[u].w += v[j].w;
                    seen[u] += 1;
                }
            }
            if (mm[u] >= M) continue;
            if (seen[u] > 1) {
                const float inv = 1.0f / (float)seen[u];
                acc[u].x *= inv; acc[u].y *= inv; acc[u].z *= inv; acc[u].w *= inv;
            }
            __stcs(a.vox_img + (size_t)mm[u] * cf4 + c, acc[u]);
            if (c == 0) a.vox_cnt[mm[u]] = seen[u];
        }
    }
}

// Mean of the p x p window of map texels that pooled texel (ty, tx) of map `map` stands for, column c:
// the same sum, in the same order, as pool_features_kernel (rows outer, columns inner, one multiply by
// the reciprocal of the texel count), so the value is the pooled map's, bit for bit.
__device__ __forceinline__ float4 window_mean(const VifArgs& a, uint32_t map, int ty, int tx, int c, int cf4) {
    const int j0 = ty * a.pool, j1 = min(a.Hf, j0 + a.pool), i0 = tx * a.pool, i1 = min(a.Wf, i0 + a.pool);
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int j = j0; j < j1; ++j) {
        const float4* row = a.feat + (((size_t)map * a.Hf + j) * a.Wf + i0) * cf4 + c;
        for (int x = 0; x < i1 - i0; ++x) {
            const float4 v = __ldg(row + (size_t)x * cf4);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
    }
    const float inv = 1.0f / (float)((j1 - j0) * (i1 - i0));
    return make_float4(s.x * inv, s.y * inv, s.z * inv, s.w * inv);
}

// gather_column on the pooled map that is never materialised: the four taps are window means.
__device__ __forceinline__ float4 pooled_column(const VifArgs& a, const uint4& rec, int c, int cf4) {
    if (rec.x == kZeroRow) return make_float4(0.f, 0.f, 0.f, 0.f);
    uint32_t t = rec.x;
    const int x0 = (int)(t % (uint32_t)a.Wp);
    t /= (uint32_t)a.Wp;
    const int y0 = (int)(t % (uint32_t)a.Hp);
    const uint32_t map = t / (uint32_t)a.Hp;
    const int x1 = x0 + (int)(rec.y & 1u), y1 = y0 + (int)((rec.y >> 1) & 1u);
    const float4 f00 = window_mean(a, map, y0, x0, c, cf4);
    const float4 f01 = x1 != x0 ? window_mean(a, map, y0, x1, c, cf4) : f00;
    const float4 f10 = y1 != y0 ? window_mean(a, map, y1, x0, c, cf4) : f00;
    const float4 f11 = y1 != y0 ? (x1 != x0 ? window_mean(a, map, y1, x1, c, cf4) : f10) : f01;
    return blend(f00, f01, f10, f11, __uint_as_float(rec.z), __uint_as_float(rec.w));
}

// vif_mean without the per-point rows: every listed point's row is blended from its four taps of
// the feature maps here (the blend of the gather stage, from the point's pixel and camera), so the
// [points, Cf] buffer is neither written nor read.  Same thread layout as vif_mean.
// kPooled: the taps are window means of the unpooled maps (emc2_voxel_image_pooled).
template <int CF4, bool kPooled>
__global__ void __launch_bounds__(CF4 > 0 ? 16 * CF4 : kThreads) vif_sample_kernel(VifArgs a) {
    if (*a.bad) return;
    const int M = voxels_in_use(a);
    const int cf4 = CF4 > 0 ? CF4 : a.cf4;
    const int rows = (int)blockDim.x / cf4;
    const int r = (int)threadIdx.x / cf4, c = (int)threadIdx.x - r * cf4;
    if (r >= rows) return;
    const uint32_t row_stride = (uint32_t)a.Wf * cf4;
    const int stride = gridDim.x * rows;
    for (int m0 = blockIdx.x * rows + r; m0 < M; m0 += 2 * stride) {
        int mm[2] = {m0, m0 + stride}, s0[2], n[2], seen[2] = {0, 0};
        float4 acc[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const bool ok = mm[u] < M;
            s0[u] = ok ? a.start[mm[u]] : 0;
            n[u] = ok ? min(a.counts[mm[u]], a.cursor[mm[u]]) : 0;   // never past what this call appended
            acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        // The first entries of the two voxels together, then the rest of each list, two at a time;
        // every voxel's rows are added in list order.
        {
            uint4 rec[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) rec[u] = n[u] > 0 ? a.recs[s0[u]] : make_uint4(kZeroRow, 0u, 0u, 0u);
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                acc[u] = kPooled ? pooled_column(a, rec[u], c, cf4) : gather_column(a.feat, rec[u], c, (uint32_t)cf4, row_stride);
                seen[u] = rec[u].x != kZeroRow ? 1 : 0;
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            for (int k = 1; k < n[u]; k += 2) {
                uint4 rec[2];
                float4 v[2];
#pragma unroll
                for (int j = 0; j < 2; ++j) rec[j] = k + j < n[u] ? a.recs[s0[u] + k + j] : make_uint4(kZeroRow, 0u, 0u, 0u);
#pragma unroll
                for (int j = 0; j < 2; ++j)
                    v[j] = kPooled ? pooled_column(a, rec[j], c, cf4) : gather_column(a.feat, rec[j], c, (uint32_t)cf4, row_stride);
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    if (rec[j].x == kZeroRow) continue;
                    acc[u].x += v[j].x; acc[u].y += v[j].y; acc[u].z += v[j].z; acc[u].w += v[j].w;
                    seen[u] += 1;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (mm[u] >= M) continue;
            if (seen[u] > 1) {
                const float inv = 1.0f / (float)seen[u];
                acc[u].x *= inv; acc[u].y *= inv; acc[u].z *= inv; acc[u].w *= inv;
            }
            __stcs(a.vox_img + (size_t)mm[u] * cf4 + c, acc[u]);
            if (c == 0) a.vox_cnt[mm[u]] = seen[u];
        }
    }
}

}  // namespace

int voxel_image_scan_max_blocks() {
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, vif_scan_kernel, kThreads, 0) != cudaSuccess) return 0;
    return sms * min(per_sm, 2);
}

// d_gathered != null: rows are read from it and d_vis_mask says which points count; else rows are
// sampled from d_feat at d_uvd in camera d_cam, and a point counts iff its camera is >= 0.
int launch_voxel_image(emc2_bridge* h, int B, int N, int capacity, const int32_t* d_point_voxel,
                       const int32_t* d_counts, const int32_t* d_num_voxels, const uint8_t* d_vis_mask,
                       const float* d_gathered, const float* d_uvd, const int8_t* d_cam, const float* d_feat,
                       float* d_vox_img, int32_t* d_vox_img_count, cudaStream_t st, int pool) {
    const emc2_config_t& cfg = h->cfg;
    VifArgs a;
    a.pv = d_point_voxel; a.counts = d_counts; a.num_voxels = d_num_voxels; a.vis = d_vis_mask;
    a.gathered = reinterpret_cast<const float4*>(d_gathered);
    a.cam = d_cam; a.uvd = d_uvd; a.feat = reinterpret_cast<const float4*>(d_feat);
    a.N = N; a.K = cfg.num_cameras; a.Hf = cfg.feat_h; a.Wf = cfg.feat_w;
    a.inv_stride = 1.0f / (float)cfg.feat_stride; a.offset = cfg.feat_offset;
    a.pool = pool; a.Hp = cfg.feat_h; a.Wp = cfg.feat_w;
    if (pool > 1) {
        // The pooled map: texel J sits at the centre of its window, (J p + (p - 1) / 2) texels of stride s in.
        a.Hp = (cfg.feat_h + pool - 1) / pool; a.Wp = (cfg.feat_w + pool - 1) / pool;
        a.inv_stride = 1.0f / ((float)cfg.feat_stride * (float)pool);
        a.offset = cfg.feat_offset + 0.5f * (float)(pool - 1) * (float)cfg.feat_stride;
    }
    a.vox_img = reinterpret_cast<float4*>(d_vox_img); a.vox_cnt = d_vox_img_count;
    a.start = h->d_vif_start; a.cursor = h->d_vif_cursor; a.list = h->d_vif_list; a.part = h->d_vif_part;
    a.recs = h->d_vif_recs;
    a.bad = h->d_vif_part + h->vif_scan_blocks;
    a.status = h->d_status;
    a.total = (long long)B * N;
    a.capacity = (int)min((long long)capacity, a.total);   // a voxel holds at least one point
    a.cf4 = cfg.feat_c / 4;
    if (a.total == 0 || a.capacity == 0) return EMC2_OK;
    if (a.cf4 > kThreads) return EMC2_ERR_INVALID_ARG;      // a feature row must fit one CTA
    {
        LaunchScope ls(h, K_VIF_SCAN, st);
        void* args[] = {&a};
        cudaError_t e = cudaLaunchCooperativeKernel((const void*)vif_scan_kernel, dim3(h->vif_scan_blocks),
                                                    dim3(kThreads), args, 0, st);
        if (e != cudaSuccess) return check_cuda(h, e);
    }
    {
        LaunchScope ls(h, K_VIF_FILL, st);
        const int blocks = (int)min((long long)h->num_sms * 16, (a.total + kThreads - 1) / kThreads);
        vif_fill_kernel<<<blocks, kThreads, 0, st>>>(a);
    }
    const int blocks = (int)min((long long)h->num_sms * 16, ((long long)a.capacity + 15) / 16);
    if (d_gathered) {
        LaunchScope ls(h, K_VIF_MEAN, st);
        switch (a.cf4) {
            case 16: vif_mean_kernel<16><<<blocks, 16 * 16, 0, st>>>(a); break;
            case 20: vif_mean_kernel<20><<<blocks, 16 * 20, 0, st>>>(a); break;
            default: vif_mean_kernel<0><<<blocks, kThreads, 0, st>>>(a); break;
        }
    } else {
        LaunchScope ls(h, K_VIF_SAMPLE, st);
        if (pool > 1) {
            vif_sample_kernel<0, true><<<blocks, kThreads, 0, st>>>(a);
        } else {
            switch (a.cf4) {
                case 16: vif_sample_kernel<16, false><<<blocks, 16 * 16, 0, st>>>(a); break;
                case 20: vif_sample_kernel<20, false><<<blocks, 16 * 20, 0, st>>>(a); break;
                default: vif_sample_kernel<0, false><<<blocks, kThreads, 0, st>>>(a); break;
            }
        }
    }
    return check_cuda(h, cudaGetLastError());
}

}  // namespace emc2
