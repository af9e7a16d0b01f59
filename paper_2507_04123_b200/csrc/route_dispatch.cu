// Stages 3 and 4 of the bridge: per-point expert id from distance and visibility buckets
// (Scenario-Adaptive Dispatcher, Sec. 3.2: near is < D, far is >= D), then a stable
// counting-sort partition of point rows and feature rows into per-expert segments whose
// offsets are exclusive prefix sums (Sec. 3.6).
//
// Three launches: (1) expert ids plus one histogram per 256-point tile, counted with warp
// ballots; (2) a small scan, one CTA per frame, that turns tile histograms into per-frame
// expert offsets and per-tile bases; (3) one CTA per tile ranks its points inside the tile with ballots and
// popcounts, writes the permutation and moves the 16/20-byte point rows and the 256/320-byte
// feature rows with coalesced 128-bit accesses.
#include <cmath>
#include <mutex>

#include "bridge_internal.cuh"

namespace emc2 {
namespace {

struct RouteArgs {
    const float* pts;
    const uint8_t* vis;
    uint8_t* expert;
    int* tile_counts;     // [B, tiles, E]
    int N, tiles, E, T;
    float thr2[EMC2_MAX_THRESHOLDS];
    uint8_t lut[16];
};

constexpr int kHistTiles = 4;         // tiles one CTA of route_hist_kernel takes (independent loads per thread)

// grid = (ceil(tiles per frame / kHistTiles), B); tiles never straddle frames.  Thread t takes
// point t of each of the CTA's tiles, so its loads are independent; one histogram per tile.
template <int C>
__global__ void __launch_bounds__(kThreads) route_hist_kernel(const __grid_constant__ RouteArgs a) {
    __shared__ int hist[kHistTiles][EMC2_MAX_EXPERTS];
    const int b = blockIdx.y, t = threadIdx.x, lane = t & 31;
    const int tile0 = blockIdx.x * kHistTiles;
    if (t < kHistTiles * EMC2_MAX_EXPERTS) hist[t / EMC2_MAX_EXPERTS][t % EMC2_MAX_EXPERTS] = 0;
    float x[kHistTiles], y[kHistTiles];
    unsigned vis[kHistTiles];
#pragma unroll
    for (int u = 0; u < kHistTiles; ++u) {
        const int i = (tile0 + u) * kTile + t;
        x[u] = y[u] = 0.0f;
        vis[u] = 0u;
        if (i < a.N) {
            const size_t gi = (size_t)b * a.N + i;
            const float2 xy = C == 4 ? *reinterpret_cast<const float2*>(a.pts + gi * 4)
                                     : make_float2(__ldg(a.pts + gi * C), __ldg(a.pts + gi * C + 1));
            x[u] = xy.x; y[u] = xy.y;
            vis[u] = a.vis[gi];
        }
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < kHistTiles; ++u) {
        const int i = (tile0 + u) * kTile + t;
        int e = -1;
        if (i < a.N) {
            const float r2 = __fmaf_rn(x[u], x[u], __fmul_rn(y[u], y[u]));
            int bucket = 0;
            for (int k = 0; k < a.T; ++k) bucket += (r2 >= a.thr2[k]) ? 1 : 0;
            e = a.lut[(vis[u] != 0u ? 8 : 0) + bucket];
            a.expert[(size_t)b * a.N + i] = (uint8_t)e;
        }
        for (int k = 0; k < a.E; ++k) {
            const unsigned m = __ballot_sync(0xFFFFFFFFu, e == k);
            if (lane == 0 && m) atomicAdd(&hist[u][k], __popc(m));
        }
    }
    __syncthreads();
    if (t < kHistTiles * EMC2_MAX_EXPERTS) {
        const int u = t / EMC2_MAX_EXPERTS, k = t % EMC2_MAX_EXPERTS;
        if (tile0 + u < a.tiles && k < a.E)
            a.tile_counts[((size_t)b * a.tiles + tile0 + u) * a.E + k] = hist[u][k];
    }
}

template <int C>
void launch_hist(const RouteArgs& ra, int B, cudaStream_t st) {
    const dim3 grid((ra.tiles + kHistTiles - 1) / kHistTiles, B);
    route_hist_kernel<C><<<grid, kThreads, 0, st>>>(ra);
}

constexpr int kScanThreads = 1024;

// One CTA of 1024 threads per frame.  Every thread owns a run of consecutive tiles and loads all
// their counts up front; per expert, a CTA-wide exclusive scan of the run totals gives the run's
// base, the expert totals give the frame's offsets, and the bases are written in one sweep.
__global__ void __launch_bounds__(kScanThreads)
route_scan_kernel(const int* __restrict__ tile_counts, int* __restrict__ tile_base, int32_t* offsets,
                  int tiles, int E, int N) {
    constexpr int kWarps = kScanThreads / 32;
    __shared__ int wsum[EMC2_MAX_EXPERTS][kWarps];
    __shared__ int etot[EMC2_MAX_EXPERTS + 1];
    const int b = blockIdx.x, t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int* cnt = tile_counts + (size_t)b * tiles * E;
    int* base = tile_base + (size_t)b * tiles * E;
    const int per = (tiles + kScanThreads - 1) / kScanThreads;
    const int lo = min(tiles, t * per), hi = min(tiles, lo + per);
    int run[EMC2_MAX_EXPERTS];            // this thread's total, then its exclusive base, per expert
#pragma unroll
    for (int e = 0; e < EMC2_MAX_EXPERTS; ++e) run[e] = 0;
    for (int i = lo; i < hi; ++i) {
#pragma unroll
        for (int e = 0; e < EMC2_MAX_EXPERTS; ++e)
            if (e < E) run[e] += cnt[(size_t)i * E + e];
    }
#pragma unroll
    for (int e = 0; e < EMC2_MAX_EXPERTS; ++e) {
        if (e >= E) break;
        int x = run[e];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xFFFFFFFFu, x, d);
            if (lane >= d) x += y;
        }
        if (lane == 31) wsum[e][warp] = x;
        run[e] = x - run[e];              // exclusive inside the warp
    }
    __syncthreads();
    if (warp < E) {                       // warp e scans the warp totals of expert e
        int x = wsum[warp][lane];
        const int v = x;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xFFFFFFFFu, x, d);
            if (lane >= d) x += y;
        }
        wsum[warp][lane] = x - v;
        if (lane == 31) etot[warp] = x;
    }
    __syncthreads();
    if (t == 0) {
        int acc = 0;
        for (int e = 0; e < E; ++e) { const int c = etot[e]; etot[e] = acc; acc += c; }
        etot[E] = acc;
    }
    __syncthreads();
    if (t <= E) offsets[(size_t)b * (E + 1) + t] = etot[t];
#pragma unroll
    for (int e = 0; e < EMC2_MAX_EXPERTS; ++e)
        if (e < E) run[e] += etot[e] + wsum[e][warp];
    for (int i = lo; i < hi; ++i) {
#pragma unroll
        for (int e = 0; e < EMC2_MAX_EXPERTS; ++e) {
            if (e < E) {
                base[(size_t)i * E + e] = run[e];
                run[e] += cnt[(size_t)i * E + e];
            }
        }
    }
}

struct ScatterArgs {
    const float* pts;
    const float4* feat;
    const uint8_t* expert;
    const int* tile_base;
    int32_t* perm;
    float* pts_out;
    float4* feat_out;
    int N, tiles, E, cf4;
};

// CF4 > 0: Cf/4 known at compile time, blockDim.x == 16 * CF4.  CF4 == 0: any Cf, 256 threads.
template <int C, int CF4>
__global__ void __launch_bounds__(CF4 > 0 ? 16 * CF4 : kThreads) dispatch_scatter_kernel(ScatterArgs a) {
    __shared__ int sdest[kTile];
    __shared__ int wcnt[kTile / 32][EMC2_MAX_EXPERTS];
    const int b = blockIdx.y, tile = blockIdx.x, t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int i0 = tile * kTile;
    const int npts = min(kTile, a.N - i0);
    const size_t f0 = (size_t)b * a.N;        // first row of the frame
    const size_t g0 = f0 + i0;
    const int cf4 = CF4 > 0 ? CF4 : a.cf4;

    // Stable rank inside the tile: ballots per expert (warps past the tile only take part in
    // the barriers).
    int e = -1, rank = 0;
    if (t < kTile) {
        e = t < npts ? (int)a.expert[g0 + t] : -1;
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
        const int d = a.tile_base[((size_t)b * a.tiles + tile) * a.E + e] + before + rank;
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
    // Feature rows: 16 rows x Cf/4 columns of threads; each thread keeps its column, reads
    // eight rows (eight independent 128-bit streaming loads), then writes them to their slots.
    const float4* fsrc = a.feat + g0 * cf4;
    float4* fdst = a.feat_out + f0 * cf4;
    if constexpr (CF4 > 0) {
        const int c = t % CF4, r0 = t / CF4;
#pragma unroll
        for (int j0 = 0; j0 < kTile / 16; j0 += 8) {
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int r = r0 + 16 * (j0 + u);
                if (r < npts) v[u] = __ldcs(fsrc + r * CF4 + c);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int r = r0 + 16 * (j0 + u);
                if (r < npts) __stcs(fdst + (size_t)sdest[r] * CF4 + c, v[u]);
            }
        }
    } else {
        const int items = npts * cf4;
        for (int i = t; i < items; i += blockDim.x) {
            const int r = i / cf4, c = i - r * cf4;
            __stcs(fdst + (size_t)sdest[r] * cf4 + c, __ldcs(fsrc + i));
        }
    }
}

template <int C>
void launch_scatter(emc2_bridge* h, const ScatterArgs& a, dim3 grid, cudaStream_t st) {
    LaunchScope ls(h, K_DISPATCH_SCATTER, st);
    switch (a.cf4) {
        case 16: dispatch_scatter_kernel<C, 16><<<grid, 16 * 16, 0, st>>>(a); break;
        case 20: dispatch_scatter_kernel<C, 20><<<grid, 16 * 20, 0, st>>>(a); break;
        default: dispatch_scatter_kernel<C, 0><<<grid, kThreads, 0, st>>>(a); break;
    }
}

}  // namespace

namespace {

struct SceneArgs {
    const int32_t* offsets;
    int32_t* scene_expert;
    int B, E, min_points;
    uint8_t priority[EMC2_MAX_EXPERTS];
};

// One thread per frame: the expert of highest priority that owns enough points (Sec. 3.2).
__global__ void scene_route_kernel(const __grid_constant__ SceneArgs a) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= a.B) return;
    const int32_t* off = a.offsets + (size_t)b * (a.E + 1);
    int best = -1, best_pr = -1;
    for (int e = 0; e < a.E; ++e) {
        const int count = off[e + 1] - off[e];
        if (count >= a.min_points && (int)a.priority[e] > best_pr) { best = e; best_pr = a.priority[e]; }
    }
    a.scene_expert[b] = best;
}

}  // namespace

int launch_scene_route(emc2_bridge* h, int B, const int32_t* d_offsets, const uint8_t* priority, int min_points,
                       int32_t* d_scene_expert, cudaStream_t st) {
    SceneArgs a;
    a.offsets = d_offsets; a.scene_expert = d_scene_expert;
    a.B = B; a.E = h->cfg.num_experts; a.min_points = min_points < 1 ? 1 : min_points;
    for (int e = 0; e < EMC2_MAX_EXPERTS; ++e) a.priority[e] = e < a.E ? priority[e] : 0;
    {
        LaunchScope ls(h, K_SCENE_ROUTE, st);
        scene_route_kernel<<<(B + 31) / 32, 32, 0, st>>>(a);
    }
    return check_cuda(h, cudaGetLastError());
}

void launch_route_scan(emc2_bridge* h, int b0, int B, int tiles, int N, int32_t* d_offsets, cudaStream_t st) {
    LaunchScope ls(h, K_ROUTE_SCAN, st);
    const size_t t0 = (size_t)b0 * tiles * h->cfg.num_experts;
    route_scan_kernel<<<B, kScanThreads, 0, st>>>(h->d_tile_counts + t0, h->d_tile_base + t0, d_offsets, tiles,
                                                  h->cfg.num_experts, N);
}

int launch_route_dispatch(emc2_bridge* h, int B, int N, const float* d_points, const uint8_t* d_vis_mask,
                          const float* d_gathered, uint8_t* d_expert, int32_t* d_offsets, int32_t* d_perm,
                          float* d_points_out, float* d_feat_out, cudaStream_t st) {
    const emc2_config_t& c = h->cfg;
    const int tiles = (N + kTile - 1) / kTile;
    const int E = c.num_experts;
    if (B == 0) return EMC2_OK;
    const dim3 grid(tiles > 0 ? tiles : 1, B);
    RouteArgs ra;
    ra.pts = d_points; ra.vis = d_vis_mask; ra.expert = d_expert; ra.tile_counts = h->d_tile_counts;
    ra.N = N; ra.tiles = tiles; ra.E = E; ra.T = c.num_thresholds;
    for (int k = 0; k < EMC2_MAX_THRESHOLDS; ++k) ra.thr2[k] = h->thr2[k];
    for (int k = 0; k < 16; ++k) ra.lut[k] = c.lut[k >> 3][k & 7];
    if (tiles > 0) {
        LaunchScope ls(h, K_ROUTE_HIST, st);
        if (c.point_floats == 4) launch_hist<4>(ra, B, st); else launch_hist<5>(ra, B, st);
    }
    {
        LaunchScope ls(h, K_ROUTE_SCAN, st);
        route_scan_kernel<<<B, kScanThreads, 0, st>>>(h->d_tile_counts, h->d_tile_base, d_offsets, tiles, E, N);
    }
    if (tiles > 0) {
        ScatterArgs sa;
        sa.pts = d_points; sa.feat = reinterpret_cast<const float4*>(d_gathered); sa.expert = d_expert;
        sa.tile_base = h->d_tile_base; sa.perm = d_perm; sa.pts_out = d_points_out;
        sa.feat_out = reinterpret_cast<float4*>(d_feat_out);
        sa.N = N; sa.tiles = tiles; sa.E = E; sa.cf4 = c.feat_c / 4;
        if (c.point_floats == 4) launch_scatter<4>(h, sa, grid, st); else launch_scatter<5>(h, sa, grid, st);
    }
    return check_cuda(h, cudaGetLastError());
}

}  // namespace emc2

// ------------------------------------------------------------------ handle-free variant
// emc2_route_dispatch_static: the same three kernels, with the tile histograms and tile bases in
// an array that is part of the library image instead of a cudaMalloc'ed slab.
namespace emc2 {
namespace {

// [0, ENTRIES): tile counts; [ENTRIES, 2*ENTRIES): tile bases.  Device code could name this
// array directly; host code may only use the address cudaGetSymbolAddress reports (the host-side
// symbol is a stand-in, not a device pointer).
static __device__ __align__(256) int g_static_route_scratch[2 * EMC2_STATIC_SCRATCH_ENTRIES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
int* g_static_ptr[kMaxDevices] = {nullptr};

// Device address of the array on `device`, which must be the current device.  Looked up once per
// device and cached.
cudaError_t static_scratch(int device, int** out) {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[device]) {
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_static_route_scratch);
        if (e != cudaSuccess) return e;
        g_static_ptr[device] = static_cast<int*>(p);
    }
    *out = g_static_ptr[device];
    return cudaSuccess;
}

bool aligned16_static(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace
}  // namespace emc2

extern "C" int emc2_route_dispatch_static(const emc2_config_t* config, int32_t B, int32_t N,
                                          const float* d_points, const uint8_t* d_vis_mask,
                                          const float* d_gathered, uint8_t* d_expert, int32_t* d_offsets,
                                          int32_t* d_perm, float* d_points_out, float* d_feat_out,
                                          void* cuda_stream) {
    using namespace emc2;
    if (!config) return EMC2_ERR_INVALID_ARG;
    const emc2_config_t& c = *config;
    // Only the fields this stage reads are checked.
    if (c.device < 0 || c.device >= kMaxDevices) return EMC2_ERR_BAD_CONFIG;
    if (c.point_floats != 4 && c.point_floats != 5) return EMC2_ERR_BAD_CONFIG;
    if (c.feat_c < 4 || (c.feat_c & 3)) return EMC2_ERR_BAD_CONFIG;
    if (c.num_thresholds < 0 || c.num_thresholds > EMC2_MAX_THRESHOLDS) return EMC2_ERR_BAD_CONFIG;
    for (int t = 0; t < c.num_thresholds; ++t) {
        if (!(c.thresholds[t] >= 0.0f) || !std::isfinite(c.thresholds[t])) return EMC2_ERR_BAD_CONFIG;
        if (t && !(c.thresholds[t] >= c.thresholds[t - 1])) return EMC2_ERR_BAD_CONFIG;
    }
    if (c.num_experts < 1 || c.num_experts > EMC2_MAX_EXPERTS) return EMC2_ERR_BAD_CONFIG;
    for (int v = 0; v < 2; ++v)
        for (int d = 0; d <= c.num_thresholds; ++d)
            if (c.lut[v][d] >= c.num_experts) return EMC2_ERR_BAD_CONFIG;
    if (B < 0 || N < 0 || B > EMC2_MAX_BATCH) return EMC2_ERR_INVALID_ARG;
    // No frame that fits the scratch area is anywhere near this long; it also keeps the tile count in range.
    if ((int64_t)N > (int64_t)EMC2_STATIC_SCRATCH_ENTRIES * kTile) return EMC2_ERR_TOO_LARGE;
    const int E = c.num_experts;
    const int tiles = (N + kTile - 1) / kTile;
    if ((int64_t)B * tiles * E > (int64_t)EMC2_STATIC_SCRATCH_ENTRIES) return EMC2_ERR_TOO_LARGE;
    if (B == 0) return EMC2_OK;
    if (!d_offsets) return EMC2_ERR_INVALID_ARG;
    if (N > 0 && (!d_points || !d_vis_mask || !d_gathered || !d_expert || !d_perm || !d_points_out ||
                  !d_feat_out))
        return EMC2_ERR_INVALID_ARG;
    if (!aligned16_static(d_points) || !aligned16_static(d_gathered) || !aligned16_static(d_feat_out))
        return EMC2_ERR_INVALID_ARG;
    if (N > 0 && (d_points_out == d_points || d_feat_out == d_gathered)) return EMC2_ERR_INVALID_ARG;

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return EMC2_ERR_CUDA;
    if (prev != c.device && cudaSetDevice(c.device) != cudaSuccess) return EMC2_ERR_CUDA;
    int rc = EMC2_OK;
    int* scratch = nullptr;
    if (static_scratch(c.device, &scratch) != cudaSuccess) rc = EMC2_ERR_CUDA;
    if (rc == EMC2_OK) {
        cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
        int* tile_counts = scratch;
        int* tile_base = scratch + EMC2_STATIC_SCRATCH_ENTRIES;
        const dim3 grid(tiles > 0 ? tiles : 1, B);
        if (tiles > 0) {
            RouteArgs ra;
            ra.pts = d_points; ra.vis = d_vis_mask; ra.expert = d_expert; ra.tile_counts = tile_counts;
            ra.N = N; ra.tiles = tiles; ra.E = E; ra.T = c.num_thresholds;
            for (int k = 0; k < EMC2_MAX_THRESHOLDS; ++k)
                ra.thr2[k] = k < c.num_thresholds ? c.thresholds[k] * c.thresholds[k] : 0.0f;
            for (int k = 0; k < 16; ++k) ra.lut[k] = c.lut[k >> 3][k & 7];
            if (c.point_floats == 4) launch_hist<4>(ra, B, st); else launch_hist<5>(ra, B, st);
        }
        route_scan_kernel<<<B, kScanThreads, 0, st>>>(tile_counts, tile_base, d_offsets, tiles, E, N);
        if (tiles > 0) {
            ScatterArgs sa;
            sa.pts = d_points; sa.feat = reinterpret_cast<const float4*>(d_gathered); sa.expert = d_expert;
            sa.tile_base = tile_base; sa.perm = d_perm; sa.pts_out = d_points_out;
            sa.feat_out = reinterpret_cast<float4*>(d_feat_out);
            sa.N = N; sa.tiles = tiles; sa.E = E; sa.cf4 = c.feat_c / 4;
            const int threads = sa.cf4 == 16 ? 256 : sa.cf4 == 20 ? 320 : kThreads;
            if (c.point_floats == 4) {
                if (sa.cf4 == 16) dispatch_scatter_kernel<4, 16><<<grid, threads, 0, st>>>(sa);
                else if (sa.cf4 == 20) dispatch_scatter_kernel<4, 20><<<grid, threads, 0, st>>>(sa);
                else dispatch_scatter_kernel<4, 0><<<grid, threads, 0, st>>>(sa);
            } else {
                if (sa.cf4 == 16) dispatch_scatter_kernel<5, 16><<<grid, threads, 0, st>>>(sa);
                else if (sa.cf4 == 20) dispatch_scatter_kernel<5, 20><<<grid, threads, 0, st>>>(sa);
                else dispatch_scatter_kernel<5, 0><<<grid, threads, 0, st>>>(sa);
            }
        }
        if (cudaGetLastError() != cudaSuccess) rc = EMC2_ERR_CUDA;
    }
    if (prev != c.device) cudaSetDevice(prev);
    return rc;
}
