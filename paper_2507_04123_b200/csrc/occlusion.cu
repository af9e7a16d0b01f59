// Depth-buffer occlusion for the "occluded / out-of-view" bucket of the dispatcher (Sec. 3.2 names
// occlusion as a cause of missing LiDAR detail; the test is the usual depth buffer).  Every camera
// image is cut into cells of cell x cell pixels.  occl_splat: every point, for every camera that
// sees it, lowers its cell's depth with one atomic min on the depth's bit pattern (depths are
// positive, so the integer order is the float order: the buffer is exact and deterministic).
// occl_test: a point is occluded in camera k iff its depth exceeds the cell's minimum by more
// than the margin.  Both kernels recompute pixel and depth with the projection's own fp32 chain.
#include "bridge_internal.cuh"

namespace emc2 {
namespace {

struct OcclArgs {
    const float* pts;
    const float* proj;
    const uint8_t* vis;
    uint32_t* zbuf;        // [B, K, Hz, Wz] depth bit patterns
    uint8_t* occ;
    uint8_t* clear;
    long long total;
    int N, K, Hz, Wz;
    float inv_cell, margin;
};

// Cell of camera k's buffer that point (x, y, z) of frame b falls into, and its depth there.
__device__ __forceinline__ size_t cell_and_depth(const OcclArgs& a, const float4* P, int b, int k, float x, float y,
                                                 float z, float& depth) {
    const float4 p0 = P[3 * k], p1 = P[3 * k + 1], p2 = P[3 * k + 2];
    const float t2 = __fmaf_rn(p2.x, x, __fmaf_rn(p2.y, y, __fmaf_rn(p2.z, z, p2.w)));
    const float t0 = __fmaf_rn(p0.x, x, __fmaf_rn(p0.y, y, __fmaf_rn(p0.z, z, p0.w)));
    const float t1 = __fmaf_rn(p1.x, x, __fmaf_rn(p1.y, y, __fmaf_rn(p1.z, z, p1.w)));
    const float u = __fdiv_rn(t0, t2), v = __fdiv_rn(t1, t2);
    // The cell size is a power of two, so the scaling is exact.
    // Inside the buffer for every pixel of the image; clamped, so that a mask that is not this batch's
    // cannot index outside it.
    const int cx = max(min((int)floorf(u * a.inv_cell), a.Wz - 1), 0), cy = max(min((int)floorf(v * a.inv_cell), a.Hz - 1), 0);
    depth = t2;
    return (((size_t)b * a.K + k) * a.Hz + cy) * a.Wz + cx;
}

template <int C, bool TEST>
__global__ void __launch_bounds__(kThreads) occl_kernel(const __grid_constant__ OcclArgs a) {
    const long long i = (long long)blockIdx.x * kThreads + threadIdx.x;
    if (i >= a.total) return;
    unsigned m = a.vis[i] & ((1u << a.K) - 1u);            // cameras the handle has
    unsigned occ = 0;
    if (m) {
        const int b = (int)(i / a.N);
        const float4* P = reinterpret_cast<const float4*>(a.proj) + (size_t)b * a.K * 3;
        const float* p = a.pts + i * C;
        const float x = __ldg(p), y = __ldg(p + 1), z = __ldg(p + 2);
        for (unsigned rest = m; rest; rest &= rest - 1) {
            const int k = __ffs(rest) - 1;
            float d;
            const size_t c = cell_and_depth(a, P, b, k, x, y, z, d);
            if (!TEST) {
                atomicMin(&a.zbuf[c], __float_as_uint(d));
            } else if (d > __fadd_rn(__uint_as_float(a.zbuf[c]), a.margin)) {
                occ |= 1u << k;
            }
        }
    }
    if (TEST) {
        a.occ[i] = (uint8_t)occ;
        a.clear[i] = (uint8_t)(m & ~occ);
    }
}

__global__ void __launch_bounds__(kThreads) occl_fill_kernel(uint32_t* zbuf, size_t n) {
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += (size_t)gridDim.x * kThreads)
        zbuf[i] = 0x7F800000u;                      // +infinity
}

}  // namespace

int launch_occlusion(emc2_bridge* h, int B, int N, const float* d_points, const float* d_proj,
                     const uint8_t* d_vis_mask, int cell, float margin, uint32_t* d_zbuf, uint8_t* d_occ_mask,
                     uint8_t* d_clear_mask, cudaStream_t st) {
    const emc2_config_t& c = h->cfg;
    OcclArgs a;
    a.pts = d_points; a.proj = d_proj; a.vis = d_vis_mask; a.zbuf = d_zbuf; a.occ = d_occ_mask; a.clear = d_clear_mask;
    a.total = (long long)B * N;
    a.N = N; a.K = c.num_cameras;
    a.Hz = (c.img_h + cell - 1) / cell; a.Wz = (c.img_w + cell - 1) / cell;
    a.inv_cell = 1.0f / (float)cell; a.margin = margin;
    const size_t nz = (size_t)B * a.K * a.Hz * a.Wz;
    {
        LaunchScope ls(h, K_OCCL_FILL, st);
        occl_fill_kernel<<<(unsigned)min((size_t)h->num_sms * 8, (nz + kThreads - 1) / kThreads), kThreads, 0, st>>>(d_zbuf, nz);
    }
    if (a.total > 0) {
        const unsigned blocks = (unsigned)((a.total + kThreads - 1) / kThreads);
        {
            LaunchScope ls(h, K_OCCL_SPLAT, st);
            if (c.point_floats == 4) occl_kernel<4, false><<<blocks, kThreads, 0, st>>>(a);
            else occl_kernel<5, false><<<blocks, kThreads, 0, st>>>(a);
        }
        {
            LaunchScope ls(h, K_OCCL_TEST, st);
            if (c.point_floats == 4) occl_kernel<4, true><<<blocks, kThreads, 0, st>>>(a);
            else occl_kernel<5, true><<<blocks, kThreads, 0, st>>>(a);
        }
    }
    return check_cuda(h, cudaGetLastError());
}

}  // namespace emc2
