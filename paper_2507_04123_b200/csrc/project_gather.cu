// Stage 2 of the bridge: LiDAR-to-camera projection with an in-frustum mask, then a bilinear
// gather from the chosen camera's channels-last feature map (Sec. 3.1; zero rows for points
// without a pixel, Fig. 5).
//
// One CTA owns a tile of 256 consecutive points.  Phase 1: one thread per point projects into
// all K cameras (fp32 fma chain and IEEE divide, so the mask is reproducible bit for bit),
// writes uvd / mask / camera, and leaves one 16-byte record per point in shared memory: the
// address of tap (y0, x0), two clamp flags and the two weights.  Phase 2: the CTA is laid out
// as 16 rows x (Cf/4) columns of threads; every thread keeps its float4 column and walks the
// tile's rows 16 at a time, so a warp's 128-bit loads and stores cover whole contiguous rows,
// no index division is needed, and each thread has 16 independent tap loads in flight.
#include "bridge_internal.cuh"

namespace emc2 {
namespace {

struct PgArgs {
    const float* pts;
    const float* proj;
    const float4* feat;
    float* uvd;
    uint8_t* vis;
    int8_t* cam;
    float4* out;
    long long total;
    int N, K, H, W, Hf, Wf, cf4;
    float min_depth, inv_stride;
};

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

// CF4 > 0: Cf/4 known at compile time, blockDim.x == 16 * CF4.  CF4 == 0: any Cf, 256 threads.
template <int C, int CF4>
__global__ void __launch_bounds__(CF4 > 0 ? 16 * CF4 : kThreads) project_gather_kernel(PgArgs a) {
    __shared__ __align__(16) float sp[kTile * C];
    __shared__ float suvd[kTile * 3];
    __shared__ uint4 srow[kTile];          // {tap (y0,x0) as a float4 index, clamp flags, wx, wy}

    const long long g0 = (long long)blockIdx.x * kTile;
    const int npts = (int)min((long long)kTile, a.total - g0);
    load_tile_f32(a.pts + g0 * C, npts * C, sp);
    __syncthreads();

    const int t = threadIdx.x;
    const int cf4 = CF4 > 0 ? CF4 : a.cf4;
    if (t < npts) {
        const float x = sp[t * C], y = sp[t * C + 1], z = sp[t * C + 2];
        const long long gi = g0 + t;
        const int b = (int)(gi / a.N);
        const float* P = a.proj + (size_t)b * a.K * 12;
        unsigned mask = 0;
        int best = -1;
        float bu = -1.0f, bv = -1.0f, bd = 0.0f, d0 = 0.0f;
        for (int k = 0; k < a.K; ++k, P += 12) {
            const float t0 = __fmaf_rn(__ldg(P + 0), x, __fmaf_rn(__ldg(P + 1), y, __fmaf_rn(__ldg(P + 2), z, __ldg(P + 3))));
            const float t1 = __fmaf_rn(__ldg(P + 4), x, __fmaf_rn(__ldg(P + 5), y, __fmaf_rn(__ldg(P + 6), z, __ldg(P + 7))));
            const float t2 = __fmaf_rn(__ldg(P + 8), x, __fmaf_rn(__ldg(P + 9), y, __fmaf_rn(__ldg(P + 10), z, __ldg(P + 11))));
            if (k == 0) d0 = t2;
            if (!(t2 > a.min_depth)) continue;
            const float u = __fdiv_rn(t0, t2), v = __fdiv_rn(t1, t2);
            const bool vis = (u >= 0.0f) && (u < (float)a.W) && (v >= 0.0f) && (v < (float)a.H);
            if (!vis) continue;
            mask |= 1u << k;
            if (best < 0) { best = k; bu = u; bv = v; bd = t2; }
        }
        if (best < 0) bd = isfinite(d0) ? d0 : 0.0f;
        suvd[t * 3] = bu; suvd[t * 3 + 1] = bv; suvd[t * 3 + 2] = bd;
        a.vis[gi] = (uint8_t)mask;
        a.cam[gi] = (int8_t)best;
        uint4 rec = make_uint4(kZeroRow, 0u, 0u, 0u);
        if (best >= 0) {
            // Texel coordinates: stride is a power of two, so the scaling is exact.
            const float fx = bu * a.inv_stride, fy = bv * a.inv_stride;
            const float flx = floorf(fx), fly = floorf(fy);
            int x0 = (int)flx, y0 = (int)fly;
            const int x1 = min(x0 + 1, a.Wf - 1), y1 = min(y0 + 1, a.Hf - 1);
            x0 = min(x0, a.Wf - 1);
            y0 = min(y0, a.Hf - 1);
            const uint32_t map = ((uint32_t)b * a.K + best) * a.Hf;
            rec.x = ((map + y0) * a.Wf + x0) * (uint32_t)cf4;
            rec.y = (uint32_t)(x1 - x0) | ((uint32_t)(y1 - y0) << 1);
            rec.z = __float_as_uint(fx - flx);
            rec.w = __float_as_uint(fy - fly);
        }
        srow[t] = rec;
    }
    __syncthreads();

    // uvd: the tile's 3*npts floats are contiguous in global memory.
    for (int i = t; i < npts * 3; i += blockDim.x) a.uvd[g0 * 3 + i] = suvd[i];

    float4* out = a.out + (size_t)g0 * cf4;
    const uint32_t dyv = (uint32_t)a.Wf * cf4;
    if (CF4 > 0) {
        const int c = t % CF4, r0 = t / CF4;
#pragma unroll 4
        for (int j = 0; j < kTile / 16; ++j) {
            const int r = r0 + 16 * j;
            if (r >= npts) break;
            const uint4 rec = srow[r];
            float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
            if (rec.x != kZeroRow) {
                const float4* p = a.feat + rec.x + c;
                const uint32_t dx = (rec.y & 1u) ? (uint32_t)CF4 : 0u, dy = (rec.y & 2u) ? dyv : 0u;
                const float4 f00 = __ldg(p), f01 = __ldg(p + dx), f10 = __ldg(p + dy), f11 = __ldg(p + dy + dx);
                o = blend(f00, f01, f10, f11, __uint_as_float(rec.z), __uint_as_float(rec.w));
            }
            __stcs(out + r * CF4 + c, o);
        }
    } else {
        const int items = npts * cf4;
        for (int i = t; i < items; i += blockDim.x) {
            const int r = i / cf4, c = i - r * cf4;
            const uint4 rec = srow[r];
            float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
            if (rec.x != kZeroRow) {
                const float4* p = a.feat + rec.x + c;
                const uint32_t dx = (rec.y & 1u) ? (uint32_t)cf4 : 0u, dy = (rec.y & 2u) ? dyv : 0u;
                const float4 f00 = __ldg(p), f01 = __ldg(p + dx), f10 = __ldg(p + dy), f11 = __ldg(p + dy + dx);
                o = blend(f00, f01, f10, f11, __uint_as_float(rec.z), __uint_as_float(rec.w));
            }
            __stcs(out + i, o);
        }
    }
}

template <int C>
void launch_c(emc2_bridge* h, const PgArgs& a, int tiles, cudaStream_t st) {
    LaunchScope ls(h, K_PROJECT_GATHER, st);
    switch (a.cf4) {
        case 16: project_gather_kernel<C, 16><<<tiles, 16 * 16, 0, st>>>(a); break;
        case 20: project_gather_kernel<C, 20><<<tiles, 16 * 20, 0, st>>>(a); break;
        default: project_gather_kernel<C, 0><<<tiles, kThreads, 0, st>>>(a); break;
    }
}

}  // namespace

int launch_project_gather(emc2_bridge* h, int B, int N, const float* d_points, const float* d_proj,
                          const float* d_feat, float* d_uvd, uint8_t* d_vis_mask, int8_t* d_cam,
                          float* d_gathered, cudaStream_t st) {
    const emc2_config_t& c = h->cfg;
    PgArgs a;
    a.pts = d_points; a.proj = d_proj; a.feat = reinterpret_cast<const float4*>(d_feat);
    a.uvd = d_uvd; a.vis = d_vis_mask; a.cam = d_cam; a.out = reinterpret_cast<float4*>(d_gathered);
    a.total = (long long)B * N;
    a.N = N; a.K = c.num_cameras; a.H = c.img_h; a.W = c.img_w; a.Hf = c.feat_h; a.Wf = c.feat_w;
    a.cf4 = c.feat_c / 4;
    a.min_depth = c.min_depth;
    a.inv_stride = 1.0f / (float)c.feat_stride;
    const int tiles = (int)((a.total + kTile - 1) / kTile);
    if (tiles == 0) return EMC2_OK;
    if (c.point_floats == 4) launch_c<4>(h, a, tiles, st); else launch_c<5>(h, a, tiles, st);
    return check_cuda(h, cudaGetLastError());
}

}  // namespace emc2
