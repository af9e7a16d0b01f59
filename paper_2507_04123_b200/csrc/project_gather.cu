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
    float min_depth, inv_stride, offset;
};

// Projection of one point into the K cameras of its frame (P: [K][3][4] row-major).
struct Projected {
    unsigned mask;      // bit k: visible in camera k
    int best;           // lowest visible camera, -1 if none
    float u, v, d;      // pixel and depth in `best`; (-1, -1, depth in camera 0 or 0) if none
};

// `P` points to the frame's matrices as float4 rows in shared memory.  The visibility decision is
// the one of the plain definition (fp32 fma chains, IEEE divide, compare), but the divide is only
// executed where it can matter: comparing the numerators with bounds scaled by the depth settles
// every pixel that is not within 0.01 px of an image edge, and only the chosen camera's (u, v) is
// divided out.  A warp of scattered points therefore does not walk the divide once per camera.
__device__ __forceinline__ Projected project_point(const float4* P, int K, float x, float y, float z,
                                                    int W, int H, float min_depth) {
    Projected r;
    r.mask = 0u; r.best = -1; r.u = -1.0f; r.v = -1.0f; r.d = 0.0f;
    float d0 = 0.0f, b0 = 0.0f, b1 = 0.0f;
    const float fw = (float)W, fh = (float)H;
    for (int k = 0; k < K; ++k) {
        const float4 p0 = P[3 * k], p1 = P[3 * k + 1], p2 = P[3 * k + 2];
        const float t2 = __fmaf_rn(p2.x, x, __fmaf_rn(p2.y, y, __fmaf_rn(p2.z, z, p2.w)));
        const float t0 = __fmaf_rn(p0.x, x, __fmaf_rn(p0.y, y, __fmaf_rn(p0.z, z, p0.w)));
        const float t1 = __fmaf_rn(p1.x, x, __fmaf_rn(p1.y, y, __fmaf_rn(p1.z, z, p1.w)));
        if (k == 0) d0 = t2;
        const bool front = t2 > min_depth;        // false for NaN
        // 0.001 < u < W - 0.01 and the like, multiplied through by the (positive) depth.
        const float lo = t2 * 1e-3f, hx = t2 * (fw - 1e-2f), hy = t2 * (fh - 1e-2f);
        const float ox = t2 * (fw + 1e-2f), oy = t2 * (fh + 1e-2f);
        const bool in_sure = (t0 > lo) && (t0 < hx) && (t1 > lo) && (t1 < hy);
        const bool out_sure = (t0 < -lo) || (t0 > ox) || (t1 < -lo) || (t1 > oy);
        bool vis = front && in_sure;
        if (front && !in_sure && !out_sure) {     // within a hair of an edge, or not finite: decide exactly
            const float u = __fdiv_rn(t0, t2), v = __fdiv_rn(t1, t2);
            vis = (u >= 0.0f) && (u < fw) && (v >= 0.0f) && (v < fh);
        }
        if (vis) {
            r.mask |= 1u << k;
            if (r.best < 0) { r.best = k; b0 = t0; b1 = t1; r.d = t2; }
        }
    }
    if (r.best >= 0) {
        r.u = __fdiv_rn(b0, r.d);
        r.v = __fdiv_rn(b1, r.d);
    } else {
        r.d = isfinite(d0) ? d0 : 0.0f;
    }
    return r;
}

// Copies the K 3x4 matrices of frame b into shared memory (K * 3 float4 rows).
__device__ __forceinline__ void load_proj(const float* __restrict__ proj, int b, int K, float4* sP) {
    const float4* src = reinterpret_cast<const float4*>(proj) + (size_t)b * K * 3;
    for (int i = threadIdx.x; i < K * 3; i += blockDim.x) sP[i] = __ldg(src + i);
}

// CF4 > 0: Cf/4 known at compile time, blockDim.x == 16 * CF4.  CF4 == 0: any Cf, 256 threads.
template <int C, int CF4>
__global__ void __launch_bounds__(CF4 > 0 ? 16 * CF4 : kThreads) project_gather_kernel(PgArgs a) {
    __shared__ __align__(16) float sp[kTile * C];
    __shared__ float suvd[kTile * 3];
    __shared__ uint4 srow[kTile];          // {tap (y0,x0) as a float4 index, clamp flags, wx, wy}
    __shared__ float4 sP[2][EMC2_MAX_CAMERAS * 3];   // matrices of the (at most two, if N >= 256) frames of the tile

    const long long g0 = (long long)blockIdx.x * kTile;
    const int npts = (int)min((long long)kTile, a.total - g0);
    load_tile_f32(a.pts + g0 * C, npts * C, sp);
    const int bfirst = (int)(g0 / a.N);
    const int nframes = (int)((g0 + npts - 1) / a.N) - bfirst + 1;
    if (nframes <= 2) {
        load_proj(a.proj, bfirst, a.K, sP[0]);
        if (nframes == 2) load_proj(a.proj, bfirst + 1, a.K, sP[1]);
    }
    __syncthreads();

    const int t = threadIdx.x;
    const int cf4 = CF4 > 0 ? CF4 : a.cf4;
    if (t < npts) {
        const float x = sp[t * C], y = sp[t * C + 1], z = sp[t * C + 2];
        const long long gi = g0 + t;
        const int b = (int)(gi / a.N);
        // Tiny frames (N < 256) can put more than two frames in a tile: read those from global memory.
        const float4* P = nframes <= 2 ? sP[b - bfirst] : reinterpret_cast<const float4*>(a.proj) + (size_t)b * a.K * 3;
        const Projected pr = project_point(P, a.K, x, y, z, a.W, a.H, a.min_depth);
        suvd[t * 3] = pr.u; suvd[t * 3 + 1] = pr.v; suvd[t * 3 + 2] = pr.d;
        a.vis[gi] = (uint8_t)pr.mask;
        a.cam[gi] = (int8_t)pr.best;
        const uint4 rec = tap_record(b, pr.best, pr.u, pr.v, a.K, a.Hf, a.Wf, cf4, a.inv_stride, a.offset);
        srow[t] = rec;
    }
    __syncthreads();

    // uvd: the tile's 3*npts floats are contiguous in global memory.
    for (int i = t; i < npts * 3; i += blockDim.x) a.uvd[g0 * 3 + i] = suvd[i];

    float4* out = a.out + (size_t)g0 * cf4;
    const uint32_t dyv = (uint32_t)a.Wf * cf4;
    if constexpr (CF4 > 0) {
        const int c = t % CF4, r0 = t / CF4;
#pragma unroll 4
        for (int j = 0; j < kTile / 16; ++j) {
            const int r = r0 + 16 * j;
            if (r >= npts) break;
            __stcs(out + r * CF4 + c, gather_column(a.feat, srow[r], c, (uint32_t)CF4, dyv));
        }
    } else {
        const int items = npts * cf4;
        for (int i = t; i < items; i += blockDim.x) {
            const int r = i / cf4, c = i - r * cf4;
            __stcs(out + i, gather_column(a.feat, srow[r], c, (uint32_t)cf4, dyv));
        }
    }
}

// ------------------------------------------------------------------ stages 2 - 4 in one pass
// The one-call path (emc2_bridge_run) does not send the gathered rows through memory twice.
//   project_route   per 256-point tile of a frame: projection, mask, camera, uvd, and - since the
//                   mask is now known - the expert id and the tile's expert histogram.
//   route_scan      tile histograms -> frame offsets and tile bases (shared with the staged path).
//   gather_scatter  per tile: stable rank of every point inside its expert's segment, then each
//                   feature row is blended once and stored twice, at its own row of `gathered`
//                   and at its slot of `feat_out`; point rows and the permutation go along.
// Outputs are those of the staged calls, bit for bit.
struct PrArgs {
    const float* pts;
    const float* proj;
    float* uvd;
    uint8_t* vis;
    int8_t* cam;
    uint8_t* expert;
    int* tile_counts;     // [B, tiles, E]
    int N, tiles, K, H, W;
    float min_depth;
    RouteParams rp;
    int frame0;           // kMark: frame index (in the whole batch) of this launch's first frame
    ScaleDev s0, s1;      // kMark: the voxel grids whose cells the points mark
    float4* bev;          // kMark: BEV image to zero (bev_n4 float4), or null
    size_t bev_n4;
};

// grid = (tiles per frame, B); tiles never straddle frames.  kMark: the kernel also does the
// voxelizer's marking pass (every point marks its cell in both scales' stores, and the BEV image
// is zeroed, spread over the grid), so that stage 1 starts from marked stores and reads the
// points once less; the reductions are fire-and-forget and land while the projection computes.
template <int C, bool kMark>
__global__ void __launch_bounds__(kThreads) project_route_kernel(const __grid_constant__ PrArgs a) {
    __shared__ float suvd[kTile * 3];
    __shared__ int hist[EMC2_MAX_EXPERTS];
    __shared__ float4 sP[EMC2_MAX_CAMERAS * 3];
    const int b = blockIdx.y, tile = blockIdx.x, t = threadIdx.x, lane = t & 31;
    load_proj(a.proj, b, a.K, sP);
    const int i0 = tile * kTile;
    const int npts = min(kTile, a.N - i0);
    const size_t g0 = (size_t)b * a.N + i0;
    if (t < EMC2_MAX_EXPERTS) hist[t] = 0;
    __syncthreads();
    int e = -1;
    if (t < npts) {
        const float* p = a.pts + (g0 + t) * C;
        float x, y, z;
        if (C == 4) {
            const float4 q = __ldg(reinterpret_cast<const float4*>(p));
            x = q.x; y = q.y; z = q.z;
        } else {
            x = __ldg(p); y = __ldg(p + 1); z = __ldg(p + 2);
        }
        if (kMark) mark_point(a.s0, a.s1, x, y, z, a.frame0 + b);
        const Projected pr = project_point(sP, a.K, x, y, z, a.W, a.H, a.min_depth);
        suvd[t * 3] = pr.u; suvd[t * 3 + 1] = pr.v; suvd[t * 3 + 2] = pr.d;
        a.vis[g0 + t] = (uint8_t)pr.mask;
        a.cam[g0 + t] = (int8_t)pr.best;
        const float r2 = __fmaf_rn(x, x, __fmul_rn(y, y));
        int bucket = 0;
        for (int k = 0; k < a.rp.T; ++k) bucket += (r2 >= a.rp.thr2[k]) ? 1 : 0;
        e = a.rp.lut[(pr.mask != 0u ? 8 : 0) + bucket];
        a.expert[g0 + t] = (uint8_t)e;
    }
    __syncthreads();
    for (int i = t; i < npts * 3; i += kThreads) a.uvd[g0 * 3 + i] = suvd[i];
    for (int k = 0; k < a.rp.E; ++k) {
        const unsigned m = __ballot_sync(0xFFFFFFFFu, e == k);
        if (lane == 0 && m) atomicAdd(&hist[k], __popc(m));
    }
    __syncthreads();
    if (t < a.rp.E) a.tile_counts[((size_t)b * a.tiles + tile) * a.rp.E + t] = hist[t];
    if (kMark && a.bev) {
        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        const size_t cta = (size_t)blockIdx.y * gridDim.x + blockIdx.x, nthreads = (size_t)gridDim.x * gridDim.y * kThreads;
        for (size_t i = cta * kThreads + t; i < a.bev_n4; i += nthreads) __stcs(a.bev + i, z);
    }
}

struct GsArgs {
    const float* pts;
    const float* uvd;
    const int8_t* cam;
    const uint8_t* expert;
    const int* tile_base;     // [B, tiles, E]
    const float4* feat;
    int32_t* perm;
    float* pts_out;
    float4* gathered;
    float4* feat_out;
    int N, tiles, E, K, Hf, Wf, cf4;
    float inv_stride, offset;
};

// CF4 > 0: Cf/4 known at compile time, blockDim.x == 16 * CF4.  CF4 == 0: any Cf, 256 threads.
template <int C, int CF4>
__global__ void __launch_bounds__(CF4 > 0 ? 16 * CF4 : kThreads) gather_scatter_kernel(const __grid_constant__ GsArgs a) {
    __shared__ uint4 srow[kTile];
    __shared__ int sdest[kTile];
    __shared__ int wcnt[kTile / 32][EMC2_MAX_EXPERTS];
    const int b = blockIdx.y, tile = blockIdx.x, t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int i0 = tile * kTile;
    const int npts = min(kTile, a.N - i0);
    const size_t f0 = (size_t)b * a.N;        // first row of the frame
    const size_t g0 = f0 + i0;
    const int cf4 = CF4 > 0 ? CF4 : a.cf4;
    // The tile's bases are requested first, together with the points' records: nothing below waits for
    // a second round trip to memory before the rows start to move.
    __shared__ int tbase[EMC2_MAX_EXPERTS];
    if (t >= (int)blockDim.x - EMC2_MAX_EXPERTS) {
        const int k = t - ((int)blockDim.x - EMC2_MAX_EXPERTS);
        if (k < a.E) tbase[k] = a.tile_base[((size_t)b * a.tiles + tile) * a.E + k];
    }

    // Stable rank inside the tile by ballots per expert, and the tap record of every point.
    int e = -1, rank = 0;
    if (t < kTile) {
        if (t < npts) {
            e = (int)a.expert[g0 + t];
            const float u = a.uvd[(g0 + t) * 3], v = a.uvd[(g0 + t) * 3 + 1];
            srow[t] = tap_record(b, (int)a.cam[g0 + t], u, v, a.K, a.Hf, a.Wf, cf4, a.inv_stride, a.offset);
        }
        for (int k = 0; k < a.E; ++k) {
            const unsigned m = __ballot_sync(0xFFFFFFFFu, e == k);
            if (e == k) rank = __popc(m & ((1u << lane) - 1u));
            if (lane == 0) wcnt[warp][k] = __popc(m);
        }
    }
    __syncthreads();
    if (t < npts) {
        int before = 0;
        for (int w = 0; w < warp; ++w) before += wcnt[w][e];
        const int d = tbase[e] + before + rank;
        sdest[t] = d;
        a.perm[f0 + d] = i0 + t;
    }
    __syncthreads();

    // Point rows: the tile's source floats are contiguous.
    const float* psrc = a.pts + g0 * C;
    float* pdst = a.pts_out + f0 * C;
    for (int i = t; i < npts * C; i += blockDim.x) {
        const int r = i / C, c = i - r * C;
        pdst[(size_t)sdest[r] * C + c] = __ldg(psrc + i);
    }
    // Feature rows: 16 rows x Cf/4 columns of threads; blended once, stored at both places (the
    // rows in point order only if the caller wants them).
    const bool keep = a.gathered != nullptr;
    float4* out = a.gathered + g0 * cf4;
    float4* fdst = a.feat_out + f0 * cf4;
    const uint32_t dyv = (uint32_t)a.Wf * cf4;
    if constexpr (CF4 > 0) {
        const int c = t % CF4, r0 = t / CF4;
#pragma unroll 4
        for (int j = 0; j < kTile / 16; ++j) {
            const int r = r0 + 16 * j;
            if (r >= npts) break;
            const float4 o = gather_column(a.feat, srow[r], c, (uint32_t)CF4, dyv);
            if (keep) __stcs(out + r * CF4 + c, o);
            __stcs(fdst + (size_t)sdest[r] * CF4 + c, o);
        }
    } else {
        const int items = npts * cf4;
        for (int i = t; i < items; i += blockDim.x) {
            const int r = i / cf4, c = i - r * cf4;
            const float4 o = gather_column(a.feat, srow[r], c, (uint32_t)cf4, dyv);
            if (keep) __stcs(out + i, o);
            __stcs(fdst + (size_t)sdest[r] * cf4 + c, o);
        }
    }
}

// ---- the same pass with the rows staged in shared memory and written by bulk asynchronous copies
// A thread of gather_scatter_kernel issues, per 16 bytes of output, four 128-bit tap loads and two
// 128-bit global stores; the load/store path of the SM is its busiest unit.  Here the blended
// values go to shared memory instead, a sub-tile of 32 rows at a time (the rows of one warp of the
// ranking phase), once in point order and once ordered by expert.  The first copy is one contiguous
// block of `gathered`; in the second, the rows of one expert are one contiguous run of `feat_out`
// (ranks inside a tile are stable and tile bases are prefix sums), so a sub-tile leaves as at most
// 1 + E bulk copies (cp.async.bulk shared -> global) issued by one warp, and the global stores no
// longer pass through the threads' load/store instructions.  Two stage buffers: the copies of one
// sub-tile run while the next is blended.
__device__ __forceinline__ void bulk_store(void* gdst, const void* ssrc, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 :: "l"(gdst), "r"((uint32_t)__cvta_generic_to_shared(ssrc)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Waits until at most `kPending` of this thread's bulk groups still read their shared-memory source.
template <int kPending>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" :: "n"(kPending) : "memory");
}
// Makes this thread's earlier shared-memory writes visible to the asynchronous copy engine.
__device__ __forceinline__ void fence_async_shared() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// kBoth: also stage and bulk-copy the rows in point order; otherwise those are stored from registers.
template <int C, int CF4, bool kBoth>
__global__ void __launch_bounds__(16 * CF4) gather_scatter_bulk_kernel(const __grid_constant__ GsArgs a) {
    constexpr int kSub = 32, kBufs = 2, kWarpsTile = kTile / 32;
    __shared__ __align__(128) float4 stage[kBufs][kBoth ? 2 : 1][kSub * CF4];   // [buffer][expert order, point order]
    __shared__ uint4 srow[kTile];
    __shared__ int sdest[kTile];
    __shared__ uint8_t spos[kTile];                       // row's place in its sub-tile when ordered by expert
    __shared__ int wcnt[kWarpsTile][EMC2_MAX_EXPERTS];    // rows of expert k in sub-tile w
    __shared__ int wrow[kWarpsTile][EMC2_MAX_EXPERTS];    // first feat_out row (in the frame) of that run
    const int b = blockIdx.y, tile = blockIdx.x, t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int i0 = tile * kTile;
    const int npts = min(kTile, a.N - i0);
    const size_t f0 = (size_t)b * a.N;
    const size_t g0 = f0 + i0;
    __shared__ int tbase[EMC2_MAX_EXPERTS];
    if (t >= (int)blockDim.x - EMC2_MAX_EXPERTS) {
        const int k = t - ((int)blockDim.x - EMC2_MAX_EXPERTS);
        if (k < a.E) tbase[k] = a.tile_base[((size_t)b * a.tiles + tile) * a.E + k];
    }

    int e = -1, rank = 0;
    if (t < kTile) {
        if (t < npts) {
            e = (int)a.expert[g0 + t];
            const float u = a.uvd[(g0 + t) * 3], v = a.uvd[(g0 + t) * 3 + 1];
            srow[t] = tap_record(b, (int)a.cam[g0 + t], u, v, a.K, a.Hf, a.Wf, CF4, a.inv_stride, a.offset);
        }
        for (int k = 0; k < a.E; ++k) {
            const unsigned m = __ballot_sync(0xFFFFFFFFu, e == k);
            if (e == k) rank = __popc(m & ((1u << lane) - 1u));
            if (lane == 0) wcnt[warp][k] = __popc(m);
        }
    }
    __syncthreads();
    if (t < npts) {
        int before = 0, below = 0;
        for (int w = 0; w < warp; ++w) before += wcnt[w][e];
        for (int k = 0; k < e; ++k) below += wcnt[warp][k];
        const int d = tbase[e] + before + rank;
        sdest[t] = d;
        spos[t] = (uint8_t)(below + rank);
        a.perm[f0 + d] = i0 + t;
    }
    if (t < kWarpsTile * a.E) {
        const int w = t / a.E, k = t - w * a.E;
        int before = 0;
        for (int w2 = 0; w2 < w; ++w2) before += wcnt[w2][k];
        wrow[w][k] = tbase[k] + before;
    }
    __syncthreads();

    const float* psrc = a.pts + g0 * C;
    float* pdst = a.pts_out + f0 * C;
    for (int i = t; i < npts * C; i += blockDim.x) {
        const int r = i / C, c = i - r * C;
        pdst[(size_t)sdest[r] * C + c] = __ldg(psrc + i);
    }

    const bool keep = a.gathered != nullptr;
    float4* out = a.gathered + g0 * CF4;
    float4* fdst = a.feat_out + f0 * CF4;
    const uint32_t dyv = (uint32_t)a.Wf * CF4;
    const int c = t % CF4, r0 = t / CF4;
    const int nsub = (npts + kSub - 1) / kSub;
    for (int s = 0; s < nsub; ++s) {
        const int buf = s & 1;
        if (s >= kBufs) {                                 // the copies that read this buffer must have read it
            if (warp == 0) bulk_wait_read<kBufs - 1>();
            __syncthreads();
        }
        const int nr = min(kSub, npts - s * kSub);
#pragma unroll
        for (int jj = 0; jj < kSub / 16; ++jj) {
            const int rl = r0 + 16 * jj;
            if (rl < nr) {
                const int r = s * kSub + rl;
                const float4 o = gather_column(a.feat, srow[r], c, (uint32_t)CF4, dyv);
                stage[buf][0][(int)spos[r] * CF4 + c] = o;
                if (kBoth) { if (keep) stage[buf][kBoth ? 1 : 0][rl * CF4 + c] = o; }
                else if (keep) __stcs(out + r * CF4 + c, o);
            }
        }
        fence_async_shared();
        __syncthreads();
        if (warp == 0) {
            if (lane < a.E) {
                const int cnt = wcnt[s][lane];
                int start = 0;
                for (int k = 0; k < lane; ++k) start += wcnt[s][k];
                if (cnt > 0)
                    bulk_store(fdst + (size_t)wrow[s][lane] * CF4, &stage[buf][0][start * CF4], (uint32_t)cnt * CF4 * 16u);
            } else if (kBoth && lane == 31 && keep) {
                bulk_store(out + (size_t)s * kSub * CF4, &stage[buf][kBoth ? 1 : 0][0], (uint32_t)nr * CF4 * 16u);
            }
            bulk_commit();
        }
    }
    if (warp == 0) bulk_wait_read<0>();                   // shared memory must outlive the copies that read it
}

// ---- the same pass with 256-bit accesses (sm_100: ld/st.global.v8.f32)
// A thread owns eight channels of a row instead of four: half as many load and store instructions
// (and requests into the SM's memory pipeline) per byte moved, 32 rows x Cf/8 columns per round.
// Needs Cf a multiple of 8 and 32-byte aligned maps and row buffers (checked at launch).
struct F8 { float v[8]; };

__device__ __forceinline__ F8 ldg8(const float* p) {
    F8 r;
    asm volatile("ld.global.nc.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7])
                 : "l"(p));
    return r;
}
__device__ __forceinline__ void stcs8(float* p, const F8& r) {
    asm volatile("st.global.cs.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "f"(r.v[0]), "f"(r.v[1]), "f"(r.v[2]), "f"(r.v[3]), "f"(r.v[4]), "f"(r.v[5]), "f"(r.v[6]), "f"(r.v[7])
                 : "memory");
}

// Blended channels [8c, 8c + 8) of the row described by `rec` (zeros for kZeroRow); same arithmetic as blend().
__device__ __forceinline__ F8 gather_column8(const float* __restrict__ feat, const uint4& rec, int c, uint32_t cf4,
                                             uint32_t row_stride) {
    F8 o;
#pragma unroll
    for (int k = 0; k < 8; ++k) o.v[k] = 0.f;
    if (rec.x != kZeroRow) {
        const float* p = feat + ((size_t)rec.x << 2) + 8 * c;
        const size_t dx = (rec.y & 1u) ? (size_t)cf4 * 4 : 0, dy = (rec.y & 2u) ? (size_t)row_stride * 4 : 0;
        const F8 f00 = ldg8(p), f01 = ldg8(p + dx), f10 = ldg8(p + dy), f11 = ldg8(p + dy + dx);
        const float wx = __uint_as_float(rec.z), wy = __uint_as_float(rec.w);
        const float ax = 1.0f - wx, ay = 1.0f - wy;
#pragma unroll
        for (int k = 0; k < 8; ++k)
            o.v[k] = ay * (ax * f00.v[k] + wx * f01.v[k]) + wy * (ax * f10.v[k] + wx * f11.v[k]);
    }
    return o;
}

template <int C, int CF8>
__global__ void __launch_bounds__(32 * CF8) gather_scatter_wide_kernel(const __grid_constant__ GsArgs a) {
    __shared__ uint4 srow[kTile];
    __shared__ int sdest[kTile];
    __shared__ int wcnt[kTile / 32][EMC2_MAX_EXPERTS];
    __shared__ int tbase[EMC2_MAX_EXPERTS];
    const int b = blockIdx.y, tile = blockIdx.x, t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int i0 = tile * kTile;
    const int npts = min(kTile, a.N - i0);
    const size_t f0 = (size_t)b * a.N;
    const size_t g0 = f0 + i0;
    constexpr int CF4 = 2 * CF8;
    if (t >= (int)blockDim.x - EMC2_MAX_EXPERTS) {
        const int k = t - ((int)blockDim.x - EMC2_MAX_EXPERTS);
        if (k < a.E) tbase[k] = a.tile_base[((size_t)b * a.tiles + tile) * a.E + k];
    }
    int e = -1, rank = 0;
    if (t < kTile) {
        if (t < npts) {
            e = (int)a.expert[g0 + t];
            const float u = a.uvd[(g0 + t) * 3], v = a.uvd[(g0 + t) * 3 + 1];
            srow[t] = tap_record(b, (int)a.cam[g0 + t], u, v, a.K, a.Hf, a.Wf, CF4, a.inv_stride, a.offset);
        }
        for (int k = 0; k < a.E; ++k) {
            const unsigned m = __ballot_sync(0xFFFFFFFFu, e == k);
            if (e == k) rank = __popc(m & ((1u << lane) - 1u));
            if (lane == 0) wcnt[warp][k] = __popc(m);
        }
    }
    __syncthreads();
    if (t < npts) {
        int before = 0;
        for (int w = 0; w < warp; ++w) before += wcnt[w][e];
        const int d = tbase[e] + before + rank;
        sdest[t] = d;
        a.perm[f0 + d] = i0 + t;
    }
    __syncthreads();
    const float* psrc = a.pts + g0 * C;
    float* pdst = a.pts_out + f0 * C;
    for (int i = t; i < npts * C; i += blockDim.x) {
        const int r = i / C, c = i - r * C;
        pdst[(size_t)sdest[r] * C + c] = __ldg(psrc + i);
    }
    const bool keep = a.gathered != nullptr;
    float* out = reinterpret_cast<float*>(a.gathered) + g0 * (size_t)(8 * CF8);
    float* fdst = reinterpret_cast<float*>(a.feat_out) + f0 * (size_t)(8 * CF8);
    const float* feat = reinterpret_cast<const float*>(a.feat);
    const uint32_t dyv = (uint32_t)a.Wf * CF4;
    const int c = t % CF8, r0 = t / CF8;
#pragma unroll 2
    for (int j = 0; j < kTile / 32; ++j) {
        const int r = r0 + 32 * j;
        if (r >= npts) break;
        const F8 o = gather_column8(feat, srow[r], c, (uint32_t)CF4, dyv);
        if (keep) stcs8(out + (size_t)r * (8 * CF8) + 8 * c, o);
        stcs8(fdst + (size_t)sdest[r] * (8 * CF8) + 8 * c, o);
    }
}


template <int C>
void launch_gs(emc2_bridge* h, const GsArgs& a, dim3 grid, cudaStream_t st) {
    LaunchScope ls(h, K_GATHER_SCATTER, st);
    const int mode = h->tune[EMC2_TUNE_ROW_STORE];
    if (mode == 1 && a.E < 31) {
        if (a.cf4 == 16) { gather_scatter_bulk_kernel<C, 16, true><<<grid, 16 * 16, 0, st>>>(a); return; }
        if (a.cf4 == 20) { gather_scatter_bulk_kernel<C, 20, true><<<grid, 16 * 20, 0, st>>>(a); return; }
    } else if (mode == 3 && ((reinterpret_cast<uintptr_t>(a.feat) | reinterpret_cast<uintptr_t>(a.gathered) |
                              reinterpret_cast<uintptr_t>(a.feat_out)) & 31) == 0) {
        if (a.cf4 == 16) { gather_scatter_wide_kernel<C, 8><<<grid, 32 * 8, 0, st>>>(a); return; }
        if (a.cf4 == 20) { gather_scatter_wide_kernel<C, 10><<<grid, 32 * 10, 0, st>>>(a); return; }
    } else if (mode == 2) {
        if (a.cf4 == 16) { gather_scatter_bulk_kernel<C, 16, false><<<grid, 16 * 16, 0, st>>>(a); return; }
        if (a.cf4 == 20) { gather_scatter_bulk_kernel<C, 20, false><<<grid, 16 * 20, 0, st>>>(a); return; }
    }
    switch (a.cf4) {
        case 16: gather_scatter_kernel<C, 16><<<grid, 16 * 16, 0, st>>>(a); break;
        case 20: gather_scatter_kernel<C, 20><<<grid, 16 * 20, 0, st>>>(a); break;
        default: gather_scatter_kernel<C, 0><<<grid, kThreads, 0, st>>>(a); break;
    }
}

// ------------------------------------------------------------------ planar -> channels-last
// Per map the planar data is a Cf x P matrix (P = Hf * Wf pixels) and the channels-last data its
// transpose.  A CTA moves a tile of 64 channels x 128 pixels through shared memory:
//   in   one warp per channel row, 32 consecutive pixels (128 B) per instruction;
//   out  a warp instruction covers 4 pixels x 32 channels: eight lanes store 128 contiguous bytes
//        of one pixel's row.  With a row stride of 129 words the column reads from the tile
//        (bank = channel + pixel mod 32) are conflict-free.
constexpr int kClChan = 64, kClPix = 128, kClStride = kClPix + 1;

__global__ void __launch_bounds__(256)
channels_last_kernel(const float* __restrict__ planar, float* __restrict__ last, int Cf, int P, int ptiles) {
    __shared__ float tile[kClChan][kClStride];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const size_t m = blockIdx.x / ptiles;
    const int p0 = (int)(blockIdx.x - m * ptiles) * kClPix;
    const int c0 = blockIdx.y * kClChan;
    const int nc = min(kClChan, Cf - c0);
    const float* src = planar + (m * Cf + c0) * (size_t)P + p0;
    for (int c = warp; c < nc; c += 8) {
#pragma unroll
        for (int j = 0; j < kClPix / 32; ++j) {
            const int q = lane + 32 * j;
            tile[c][q] = p0 + q < P ? __ldcs(src + (size_t)c * P + q) : 0.f;
        }
    }
    __syncthreads();
    float* dst = last + (m * P + p0) * (size_t)Cf + c0;
    const int halves = (nc + 31) / 32;                      // 32-channel halves of the tile
    const int c = 4 * (lane & 7), dq = lane >> 3;
    for (int job = warp; job < halves * (kClPix / 4); job += 8) {
        const int cc = c + 32 * (job % halves), q = 4 * (job / halves) + dq;
        if (cc >= nc || p0 + q >= P) continue;              // Cf % 4 == 0: a whole float4 or none
        const float4 v = make_float4(tile[cc][q], tile[cc + 1][q], tile[cc + 2][q], tile[cc + 3][q]);
        __stcs(reinterpret_cast<float4*>(dst + (size_t)q * Cf + cc), v);
    }
}

// ------------------------------------------------------------------ Multiscale Pooling (Sec. 3.5)
// One thread per (pooled texel, float4 column); grid = (columns of a pooled row, pooled rows,
// maps).  Consecutive threads read consecutive columns of the same input rows, so every load
// covers whole 256/320-byte rows.  Streams the maps once.
__global__ void __launch_bounds__(kThreads)
pool_features_kernel(const float4* __restrict__ feat, float4* __restrict__ pooled, int Hf, int Wf, int Hp, int Wp,
                     int cf4, int p) {
    const int ic = blockIdx.x * kThreads + threadIdx.x;     // I * cf4 + c
    if (ic >= Wp * cf4) return;
    const int I = ic / cf4, c = ic - I * cf4;
    const int J = blockIdx.y;
    const size_t m = blockIdx.z;                            // map index b * K + k
    const int j0 = J * p, j1 = min(Hf, j0 + p), i0 = I * p, i1 = min(Wf, i0 + p);
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int j = j0; j < j1; ++j) {
        const float4* row = feat + ((m * Hf + j) * Wf + i0) * cf4 + c;
#pragma unroll 4
        for (int x = 0; x < i1 - i0; ++x) {
            const float4 v = __ldcs(row + (size_t)x * cf4);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
    }
    const float inv = 1.0f / (float)((j1 - j0) * (i1 - i0));
    pooled[((m * Hp + J) * Wp) * cf4 + ic] = make_float4(s.x * inv, s.y * inv, s.z * inv, s.w * inv);
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
    a.offset = c.feat_offset;
    const int tiles = (int)((a.total + kTile - 1) / kTile);
    if (tiles == 0) return EMC2_OK;
    if (c.point_floats == 4) launch_c<4>(h, a, tiles, st); else launch_c<5>(h, a, tiles, st);
    return check_cuda(h, cudaGetLastError());
}

// Frames [b0, b0 + B) of a batch whose buffers are given whole; `bev_frames` > 0: this launch also
// zeroes the BEV image of that many frames.
int launch_project_route(emc2_bridge* h, int b0, int B, int N, const float* d_points, const float* d_proj,
                         float* d_uvd, uint8_t* d_vis_mask, int8_t* d_cam, uint8_t* d_expert, bool mark,
                         float* d_bev_to_zero, int bev_frames, cudaStream_t st) {
    const emc2_config_t& c = h->cfg;
    const int tiles = (N + kTile - 1) / kTile;
    if (B == 0 || tiles == 0) return EMC2_OK;
    const dim3 grid(tiles, B);
    const size_t p0 = (size_t)b0 * N;                      // first point of the range
    PrArgs pa;
    pa.pts = d_points + p0 * c.point_floats; pa.proj = d_proj + (size_t)b0 * c.num_cameras * 12;
    pa.uvd = d_uvd + p0 * 3; pa.vis = d_vis_mask + p0; pa.cam = d_cam + p0;
    pa.expert = d_expert + p0; pa.tile_counts = h->d_tile_counts + (size_t)b0 * tiles * c.num_experts;
    pa.N = N; pa.tiles = tiles; pa.K = c.num_cameras; pa.H = c.img_h; pa.W = c.img_w;
    pa.min_depth = c.min_depth;
    pa.rp = route_params(h);
    pa.frame0 = b0;
    pa.s0 = h->scale[0]; pa.s1 = h->scale[1];
    pa.bev = nullptr; pa.bev_n4 = 0;
    if (mark && d_bev_to_zero && bev_frames > 0) {
        const size_t bev_n = (size_t)bev_frames * c.point_floats * h->scale[1].dims[1] * h->scale[1].dims[0];
        if (bev_n & 3) {
            cudaMemsetAsync(d_bev_to_zero, 0, bev_n * sizeof(float), st);
        } else {
            pa.bev = reinterpret_cast<float4*>(d_bev_to_zero);
            pa.bev_n4 = bev_n >> 2;
        }
    }
    {
        LaunchScope ls(h, K_PROJECT_ROUTE, st);
        if (c.point_floats == 4) {
            if (mark) project_route_kernel<4, true><<<grid, kThreads, 0, st>>>(pa);
            else project_route_kernel<4, false><<<grid, kThreads, 0, st>>>(pa);
        } else {
            if (mark) project_route_kernel<5, true><<<grid, kThreads, 0, st>>>(pa);
            else project_route_kernel<5, false><<<grid, kThreads, 0, st>>>(pa);
        }
    }
    return check_cuda(h, cudaGetLastError());
}

int launch_scan_gather_scatter(emc2_bridge* h, int b0, int B, int N, const float* d_points, const float* d_feat,
                               const float* d_uvd, const int8_t* d_cam, float* d_gathered, const uint8_t* d_expert,
                               int32_t* d_offsets, int32_t* d_perm, float* d_points_out, float* d_feat_out,
                               cudaStream_t st) {
    const emc2_config_t& c = h->cfg;
    if (B == 0) return EMC2_OK;
    const int tiles = (N + kTile - 1) / kTile;
    const dim3 grid(tiles > 0 ? tiles : 1, B);
    const int E = c.num_experts;
    const size_t p0 = (size_t)b0 * N, t0 = (size_t)b0 * tiles * E;
    launch_route_scan(h, b0, B, tiles, N, d_offsets + (size_t)b0 * (E + 1), st);
    if (tiles > 0) {
        GsArgs ga;
        ga.pts = d_points + p0 * c.point_floats; ga.uvd = d_uvd + p0 * 3; ga.cam = d_cam + p0; ga.expert = d_expert + p0;
        ga.tile_base = h->d_tile_base + t0;
        ga.feat = reinterpret_cast<const float4*>(d_feat + (size_t)b0 * c.num_cameras * c.feat_h * c.feat_w * c.feat_c);
        ga.perm = d_perm + p0; ga.pts_out = d_points_out + p0 * c.point_floats;
        ga.gathered = d_gathered ? reinterpret_cast<float4*>(d_gathered + p0 * c.feat_c) : nullptr;
        ga.feat_out = reinterpret_cast<float4*>(d_feat_out + p0 * c.feat_c);
        ga.N = N; ga.tiles = tiles; ga.E = E; ga.K = c.num_cameras; ga.Hf = c.feat_h; ga.Wf = c.feat_w;
        ga.cf4 = c.feat_c / 4;
        ga.inv_stride = 1.0f / (float)c.feat_stride;
        ga.offset = c.feat_offset;
        if (c.point_floats == 4) launch_gs<4>(h, ga, grid, st); else launch_gs<5>(h, ga, grid, st);
    }
    return check_cuda(h, cudaGetLastError());
}

int launch_channels_last(emc2_bridge* h, int B, const float* d_planar, float* d_feat, cudaStream_t st) {
    const emc2_config_t& c = h->cfg;
    const long long P = (long long)c.feat_h * c.feat_w;
    const long long ptiles = (P + kClPix - 1) / kClPix;
    const long long ctas = (long long)B * c.num_cameras * ptiles;
    const int ct = (c.feat_c + kClChan - 1) / kClChan;
    if (P > 0x7FFFFFFFLL || ctas > 0x7FFFFFFFLL || ct > 65535) return EMC2_ERR_INVALID_ARG;
    LaunchScope ls(h, K_CHANNELS_LAST, st);
    const dim3 grid((unsigned)ctas, ct);
    channels_last_kernel<<<grid, 256, 0, st>>>(d_planar, d_feat, c.feat_c, (int)P, (int)ptiles);
    return check_cuda(h, cudaGetLastError());
}

int launch_pool_features(emc2_bridge* h, int B, int p, const float* d_feat, float* d_pooled, cudaStream_t st) {
    const emc2_config_t& c = h->cfg;
    const int Hp = (c.feat_h + p - 1) / p, Wp = (c.feat_w + p - 1) / p, cf4 = c.feat_c / 4;
    if (Hp > 65535) return EMC2_ERR_INVALID_ARG;           // grid limit: one pooled row per blockIdx.y
    const dim3 grid((Wp * cf4 + kThreads - 1) / kThreads, Hp, B * c.num_cameras);
    {
        LaunchScope ls(h, K_POOL_FEATURES, st);
        pool_features_kernel<<<grid, kThreads, 0, st>>>(reinterpret_cast<const float4*>(d_feat),
                                                        reinterpret_cast<float4*>(d_pooled), c.feat_h, c.feat_w, Hp,
                                                        Wp, cf4, p);
    }
    return check_cuda(h, cudaGetLastError());
}

}  // namespace emc2
