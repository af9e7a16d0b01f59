// Stage 1 of the bridge: two-scale voxelization, dedup in canonical order, per-voxel counts
// and means, BEV scatter (Sec. 3.1 preprocessing; BEV for the 2D expert of Sec. 3.3).
//
// Dedup is direct-addressed, with no sort and no hash probing.  Large grids keep one bit per
// cell: the store is an array of {32 cell bits, rank} pairs in cell order.  Grids small enough
// keep one record {point count, rank, rank among cells over the cap, -} per cell.  "Rank" is
// the number of occupied cells before this word / cell in ascending (b, z, y, x) order, which
// is the canonical voxel order, so a point finds its voxel row with ONE 8- or 16-byte load plus
// a popcount, and no sort is ever needed.
//
//   vox_mark      every point marks its two cells with one fire-and-forget reduction each;
//                 the same launch zeroes the BEV image.
//   vox_scan      one cooperative launch: counts per 8 KB tile of the store, grid barrier,
//                 then the exclusive prefix sums (the parallel prefix-sum index search of
//                 Sec. 3.6) are written into the rank fields; accumulators are cleared and the
//                 bookkeeping of cells over the cap is laid out.
//   vox_accum     every point looks its rank up, writes point_voxel and adds itself to its
//                 voxels' accumulators with two fp32 vector reductions (offsets from the cell
//                 corner, the other channels, the count).
//                 Points of cells over the cap go to per-cell lists instead.
//   vox_finalize  walks the occupied tiles of the store: one thread per word / cell writes
//                 coordinates, count, mean and the BEV cell of its voxels and puts the store
//                 back to zero; in the same launch one warp per cell over the cap keeps the
//                 `cap` lowest point indices (keep-first-by-index) and sums them in fp64.
//
// Writes and reductions that land in one 32-byte sector are served one after another by the
// L2 (about 10 ns each on B200), so nothing here funnels many points into a shared flag or
// counter: the only contended words are the cells themselves.  The cost of a call follows the
// occupied tiles, not the grid volume, except for one streaming read of the store.
#include <cooperative_groups.h>

#include "bridge_internal.cuh"

namespace cg = cooperative_groups;

namespace emc2 {
namespace {

constexpr int kStatusCapacity = 1;
constexpr int kPtsPerThread = 4;                      // independent points per thread (memory-level parallelism)
constexpr int kBigTile = kThreads * kPtsPerThread;    // points per CTA in the two per-point passes
constexpr int kOvfBlocks = 296;                       // CTAs of vox_finalize that serve cells over the cap

// Where a point's cell sits in the unique list.
struct Slot {
    int m;      // row in the unique list, -1 if the point is outside the grid
    int j;      // rank among cells over the cap, -1 if the cell is not over it
};

__device__ __forceinline__ Slot slot_of(const ScaleDev& g, uint32_t cell) {
    Slot s;
    s.m = -1; s.j = -1;
    if (cell == 0xFFFFFFFFu) return s;
    if (g.mode == MODE_BITMAP) {
        const uint2 pr = *reinterpret_cast<const uint2*>(g.store + 2 * (size_t)(cell >> 5));
        s.m = (int)(pr.y + __popc(pr.x & ((1u << (cell & 31u)) - 1u)));
    } else {
        const uint4 q = *reinterpret_cast<const uint4*>(g.store + 4 * (size_t)cell);
        s.m = (int)q.y;
        if (g.cap > 0 && (int)q.x > g.cap) s.j = (int)q.z;
    }
    return s;
}

// Exclusive scan of three counters across the CTA; CTA totals in tot[].
__device__ __forceinline__ void block_excl_scan3(int v[3], int tot[3], int (*sm)[3]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    int inc[3];
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        int x = v[k];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xFFFFFFFFu, x, d);
            if (lane >= d) x += y;
        }
        inc[k] = x;
        if (lane == 31) sm[warp][k] = x;
    }
    __syncthreads();
    if (warp == 0) {
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            int x = lane < nwarp ? sm[lane][k] : 0;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int y = __shfl_up_sync(0xFFFFFFFFu, x, d);
                if (lane >= d) x += y;
            }
            if (lane < nwarp) sm[lane][k] = x;   // inclusive over warps
        }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        const int wbase = warp ? sm[warp - 1][k] : 0;
        tot[k] = sm[nwarp - 1][k];
        v[k] = wbase + inc[k] - v[k];
    }
    __syncthreads();
}

// Sum of three counters across the CTA, result valid in every thread.
__device__ __forceinline__ void block_sum3(int v[3], int (*sm)[3]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        const int x = warp_sum(v[k]);
        if (lane == 0) sm[warp][k] = x;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        int x = 0;
        for (int w = 0; w < nwarp; ++w) x += sm[w][k];
        v[k] = x;
    }
    __syncthreads();
}

// Lower corner of cell i along one axis; both per-point and per-voxel code use this value.
__device__ __forceinline__ float cell_corner(float mn, float vs, int i) { return __fmaf_rn((float)i, vs, mn); }

// ------------------------------------------------------------------ pass 1: mark cells
template <int C>
__global__ void __launch_bounds__(kThreads)
vox_mark_kernel(const float* __restrict__ pts, long long total, int N, ScaleDev s0, ScaleDev s1,
                float4* bev, size_t bev_n4) {
    __shared__ __align__(16) float sp[kBigTile * C];
    // The BEV image is zeroed here, spread over the whole grid, so it costs no extra launch.
    if (bev) {
        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < bev_n4; i += (size_t)gridDim.x * kThreads)
            __stcs(bev + i, z);
    }
    const long long g0 = (long long)blockIdx.x * kBigTile;
    const int npts = (int)min((long long)kBigTile, total - g0);
    if (npts <= 0) return;
    load_tile_f32(pts + g0 * C, npts * C, sp);
    __syncthreads();
    const int b0 = (int)(g0 / N);
    const int i0 = (int)(g0 - (long long)b0 * N);        // index of the tile's first point in frame b0
#pragma unroll
    for (int i = 0; i < kPtsPerThread; ++i) {
        const int t = threadIdx.x + i * kThreads;
        if (t >= npts) continue;
        const float x = sp[t * C], y = sp[t * C + 1], z = sp[t * C + 2];
        const int b = b0 + (i0 + t) / N;
#pragma unroll
        for (int sc = 0; sc < 2; ++sc) {
            const ScaleDev& g = sc ? s1 : s0;
            const uint32_t cell = cell_of(g, x, y, z, b);
            if (cell == 0xFFFFFFFFu) continue;
            // Results unused: these compile to reductions, which the thread does not wait for.
            if (g.mode == MODE_BITMAP) atomicOr(&g.store[2 * (size_t)(cell >> 5)], 1u << (cell & 31u));
            else atomicAdd(&g.store[4 * (size_t)cell], 1u);
        }
    }
}

// ------------------------------------------------------------------ pass 2: ranks
struct ScanArgs {
    ScaleDev s[2];
    uint32_t ntiles_used[2];    // tiles covering this call's B frames
    int capacity[2];
    int32_t* num_voxels;
    int* status;
    int* part;                  // [gridDim.x][3] per-CTA totals
    int g0;                     // CTAs [0, g0) serve scale 0, the rest scale 1
};

// One thread owns one 32-byte sector of the store: four {bits, rank} pairs or two cell records.
struct Sector {
    uint4 a, b;
};

__device__ __forceinline__ Sector load_sector(const uint32_t* store, uint32_t tile, int t) {
    const uint4* p = reinterpret_cast<const uint4*>(store) + ((size_t)tile * kThreads + t) * 2;
    Sector s;
    s.a = p[0];
    s.b = p[1];
    return s;
}

// Occupied cells, cells over the cap and points in cells over the cap of one sector.
__device__ __forceinline__ void sector_stats(const ScaleDev& g, const Sector& s, int v[3]) {
    if (g.mode == MODE_BITMAP) {
        v[0] += __popc(s.a.x) + __popc(s.a.z) + __popc(s.b.x) + __popc(s.b.z);
    } else {
        const int n0 = (int)s.a.x, n1 = (int)s.b.x;
        v[0] += (n0 > 0) + (n1 > 0);
        if (g.cap > 0) {
            if (n0 > g.cap) { v[1] += 1; v[2] += n0; }
            if (n1 > g.cap) { v[1] += 1; v[2] += n1; }
        }
    }
}

// Cooperative launch.  Every CTA owns a contiguous range of tiles of one scale.  Phase 1 counts
// and notes which tiles hold anything; after the grid barrier every CTA adds up the totals of
// the CTAs before it; phase 2 walks the occupied tiles again and writes the ranks.
__global__ void __launch_bounds__(kThreads) vox_scan_kernel(ScanArgs a) {
    __shared__ int sm[kThreads / 32][3];
    cg::grid_group grid = cg::this_grid();
    const int sc = (int)blockIdx.x >= a.g0 ? 1 : 0;
    const int first = sc ? a.g0 : 0;
    const int cta = (int)blockIdx.x - first;
    const int ncta = sc ? (int)gridDim.x - a.g0 : a.g0;
    const ScaleDev& g = a.s[sc];
    const uint32_t ntiles = a.ntiles_used[sc];
    const uint32_t per = (ntiles + (uint32_t)ncta - 1u) / (uint32_t)ncta;
    const uint32_t lo = min(ntiles, (uint32_t)cta * per), hi = min(ntiles, lo + per);
    const int t = threadIdx.x;

    int s[3] = {0, 0, 0};
    for (uint32_t tile = lo; tile < hi; ++tile) {
        const int before = s[0];
        sector_stats(g, load_sector(g.store, tile, t), s);
        const int any = __syncthreads_or(s[0] != before);
        if (t == 0) g.tile_flag[tile] = (uint32_t)any;
    }
    block_sum3(s, sm);
    if (t < 3) a.part[blockIdx.x * 3 + t] = s[t];
    grid.sync();

    // Totals of the CTAs before this one (same scale) and of the whole scale.
    int base[3] = {0, 0, 0}, tot[3] = {0, 0, 0};
    for (int c = t; c < ncta; c += kThreads) {
        const int* p = a.part + (size_t)(first + c) * 3;
        const int v0 = p[0], v1 = p[1], v2 = p[2];
        tot[0] += v0; tot[1] += v1; tot[2] += v2;
        if (c < cta) { base[0] += v0; base[1] += v1; base[2] += v2; }
    }
    block_sum3(base, sm);
    block_sum3(tot, sm);
    if (cta == 0 && t == 0) {
        g.totals[0] = tot[0]; g.totals[1] = tot[1]; g.totals[2] = tot[2];
        a.num_voxels[sc] = tot[0];
        if (tot[0] > a.capacity[sc]) atomicOr(a.status, kStatusCapacity);
    }
    // Clear the accumulators of the voxels found (two 16-byte halves per voxel).
    {
        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        const size_t n = 2 * (size_t)tot[0];
        for (size_t i = (size_t)cta * kThreads + t; i < n; i += (size_t)ncta * kThreads) g.acc[i] = z;
    }

    int carry[3] = {base[0], base[1], base[2]};
    for (uint32_t tile = lo; tile < hi; ++tile) {
        if (!g.tile_flag[tile]) continue;         // written by this CTA in phase 1; same for all threads
        Sector x = load_sector(g.store, tile, t);
        int run[3] = {0, 0, 0}, ttot[3];
        sector_stats(g, x, run);
        const bool mine = run[0] > 0;
        block_excl_scan3(run, ttot, sm);          // run[] = exclusive offsets inside the tile
        if (mine) {
            int m = carry[0] + run[0];
            if (g.mode == MODE_BITMAP) {
                x.a.y = (uint32_t)m; m += __popc(x.a.x);
                x.a.w = (uint32_t)m; m += __popc(x.a.z);
                x.b.y = (uint32_t)m; m += __popc(x.b.x);
                x.b.w = (uint32_t)m;
            } else {
                int j = carry[1] + run[1], off = carry[2] + run[2];
                const uint32_t cell0 = (tile * (uint32_t)kThreads + t) * 2u;
                x.a.y = (uint32_t)m; x.a.z = (uint32_t)j;
                const int n0 = (int)x.a.x, n1 = (int)x.b.x;
                if (g.cap > 0 && n0 > g.cap) {
                    g.ovf_vox[j] = m; g.ovf_off[j] = off; g.ovf_cell[j] = cell0; g.ovf_cursor[(size_t)j * kCursorStride] = 0;
                    j += 1; off += n0;
                }
                m += n0 > 0;
                x.b.y = (uint32_t)m; x.b.z = (uint32_t)j;
                if (g.cap > 0 && n1 > g.cap) {
                    g.ovf_vox[j] = m; g.ovf_off[j] = off; g.ovf_cell[j] = cell0 + 1u; g.ovf_cursor[(size_t)j * kCursorStride] = 0;
                }
            }
            uint4* p = reinterpret_cast<uint4*>(g.store) + ((size_t)tile * kThreads + t) * 2;
            p[0] = x.a;
            p[1] = x.b;
        }
        carry[0] += ttot[0]; carry[1] += ttot[1]; carry[2] += ttot[2];
    }
}

// ------------------------------------------------------------------ pass 3: accumulate
struct AccumArgs {
    ScaleDev s[2];
    uint32_t ntiles_used[2];
    int capacity[2];
    int32_t* coords[2];
    int32_t* counts[2];
    int32_t* point_voxel[2];
    float* mean[2];
    float* bev;
};

// Per-voxel accumulator, 32 bytes of fp32: {sum dx, sum dy, sum dz, sum ch3}, {sum ch4, count, -, -},
// where d* are offsets from the cell's lower corner, so that those sums stay small.  Two vector
// reductions per point and scale.  A sum of n terms carries a relative error of at most n * 2^-24
// (far less in practice, since the roundings do not line up).
template <int C>
__global__ void __launch_bounds__(kThreads)
vox_accum_kernel(const float* __restrict__ pts, long long total, int N, AccumArgs a) {
    __shared__ __align__(16) float sp[kBigTile * C];
    const long long g0 = (long long)blockIdx.x * kBigTile;
    const int npts = (int)min((long long)kBigTile, total - g0);
    load_tile_f32(pts + g0 * C, npts * C, sp);
    __syncthreads();
    const int b0 = (int)(g0 / N);
    const int i0 = (int)(g0 - (long long)b0 * N);
    // All rank lookups first, so that a thread has eight loads in flight.
    Slot slot[2][kPtsPerThread];
    int cx[2][kPtsPerThread], cy[2][kPtsPerThread], cz[2][kPtsPerThread];
#pragma unroll
    for (int i = 0; i < kPtsPerThread; ++i) {
        const int t = threadIdx.x + i * kThreads;
#pragma unroll
        for (int sc = 0; sc < 2; ++sc) {
            const ScaleDev& g = a.s[sc];
            uint32_t cell = 0xFFFFFFFFu;
            cx[sc][i] = cy[sc][i] = cz[sc][i] = 0;
            if (t < npts) {
                const float x = sp[t * C], y = sp[t * C + 1], z = sp[t * C + 2];
                const int ix = axis_cell(x, g.mn[0], g.vs[0], g.dims[0]);
                const int iy = axis_cell(y, g.mn[1], g.vs[1], g.dims[1]);
                const int iz = axis_cell(z, g.mn[2], g.vs[2], g.dims[2]);
                if ((ix | iy | iz) >= 0) {
                    const int b = b0 + (i0 + t) / N;
                    cell = (((uint32_t)b * g.dims[2] + iz) * g.dims[1] + iy) * g.dims[0] + ix;
                    cx[sc][i] = ix; cy[sc][i] = iy; cz[sc][i] = iz;
                }
            }
            slot[sc][i] = slot_of(g, cell);
        }
    }
#pragma unroll
    for (int sc = 0; sc < 2; ++sc) {
        const ScaleDev& g = a.s[sc];
        int32_t* pv = a.point_voxel[sc];
#pragma unroll
        for (int i = 0; i < kPtsPerThread; ++i) {
            const int t = threadIdx.x + i * kThreads;
            if (t >= npts) continue;
            const Slot s = slot[sc][i];
            if (s.j >= 0) {
                // Which of this cell's points survive the cap is decided per cell in
                // vox_finalize_kernel, which also writes their point_voxel entries.
                const int tk = atomicAdd(&g.ovf_cursor[(size_t)s.j * kCursorStride], 1);
                g.ovf_list[g.ovf_off[s.j] + tk] = (int)(g0 + t);
                continue;
            }
            if (pv) pv[g0 + t] = s.m;
            if (s.m < 0 || s.m >= a.capacity[sc]) continue;
            const float dx = __fsub_rn(sp[t * C], cell_corner(g.mn[0], g.vs[0], cx[sc][i]));
            const float dy = __fsub_rn(sp[t * C + 1], cell_corner(g.mn[1], g.vs[1], cy[sc][i]));
            const float dz = __fsub_rn(sp[t * C + 2], cell_corner(g.mn[2], g.vs[2], cz[sc][i]));
            float4* row = g.acc + 2 * (size_t)s.m;
            atomicAdd(row, make_float4(dx, dy, dz, sp[t * C + 3]));
            atomicAdd(reinterpret_cast<float2*>(row + 1), make_float2(C > 4 ? sp[t * C + 4] : 0.0f, 1.0f));
        }
    }
}

// ------------------------------------------------------------------ pass 4: rows, BEV, cleanup
// Writes the output rows of voxel m, whose cell is `cell`, from its accumulator.
template <int C>
__device__ __forceinline__ void write_voxel(const AccumArgs& a, int sc, const ScaleDev& g, int m, uint32_t cell,
                                            bool over) {
    if (m >= a.capacity[sc]) return;
    const float4 a0 = g.acc[2 * (size_t)m];
    const float4 a1 = g.acc[2 * (size_t)m + 1];
    uint32_t r = cell;
    const uint32_t x = r % g.dims[0]; r /= g.dims[0];
    const uint32_t y = r % g.dims[1]; r /= g.dims[1];
    const uint32_t z = r % g.dims[2]; r /= g.dims[2];
    reinterpret_cast<int4*>(a.coords[sc])[m] = make_int4((int)r, (int)z, (int)y, (int)x);
    const int n = over ? g.cap : (int)a1.y;
    a.counts[sc][m] = n;
    if (over) return;                             // mean and BEV cell come from the cell's warp
    const double inv = 1.0 / (double)n;
    float mu[C];
    mu[0] = (float)((double)cell_corner(g.mn[0], g.vs[0], (int)x) + (double)a0.x * inv);
    mu[1] = (float)((double)cell_corner(g.mn[1], g.vs[1], (int)y) + (double)a0.y * inv);
    mu[2] = (float)((double)cell_corner(g.mn[2], g.vs[2], (int)z) + (double)a0.z * inv);
    mu[3] = (float)((double)a0.w * inv);
    if (C > 4) mu[4] = (float)((double)a1.x * inv);
    float* row = a.mean[sc] + (size_t)m * C;
#pragma unroll
    for (int k = 0; k < C; ++k) row[k] = mu[k];
    if (sc == 1 && a.bev) {
        const size_t plane = (size_t)g.dims[1] * g.dims[0];
        float* dst = a.bev + (size_t)r * C * plane + (size_t)y * g.dims[0] + x;
#pragma unroll
        for (int k = 0; k < C; ++k) dst[(size_t)k * plane] = mu[k];
    }
}

// CTAs [0, ovf_blocks) serve cells over the cap, one warp per cell: the `cap` lowest point
// indices are kept (keep-first-by-index), summed in fp64 and written as the voxel's mean; all of
// the cell's points get their point_voxel entry.  The other CTAs stride over the occupied tiles
// of both stores, one thread per word / cell: coordinates from the cell id, count, mean, BEV
// cell; then the word / cell goes back to zero.
template <int C>
__global__ void __launch_bounds__(kThreads)
vox_finalize_kernel(const float* __restrict__ pts, long long total, AccumArgs a, int ovf_blocks) {
    if ((int)blockIdx.x < ovf_blocks) {
        const int lane = threadIdx.x & 31;
        const int warp = (blockIdx.x * kThreads + threadIdx.x) >> 5;
        const int nwarps = (ovf_blocks * kThreads) >> 5;
        for (int sc = 0; sc < 2; ++sc) {
            const ScaleDev& g = a.s[sc];
            if (g.cap <= 0) continue;
            const int novf = g.totals[1];
            int32_t* pv = a.point_voxel[sc];
            for (int j = warp; j < novf; j += nwarps) {
                const int m = g.ovf_vox[j];
                const int n = g.ovf_cursor[(size_t)j * kCursorStride];
                const int* list = g.ovf_list + g.ovf_off[j];
                // Smallest index value v with #{list <= v} >= cap, by bisection on the value.
                long long lo = -1, hi = total - 1;
                while (hi - lo > 1) {
                    const long long mid = lo + (hi - lo) / 2;
                    int c = 0;
                    for (int i = lane; i < n; i += 32) c += list[i] <= mid;
                    c = warp_sum(c);
                    if (c >= g.cap) hi = mid; else lo = mid;
                }
                double acc[C];
#pragma unroll
                for (int k = 0; k < C; ++k) acc[k] = 0.0;
                for (int i = lane; i < n; i += 32) {
                    const int v = list[i];
                    const bool keep = v <= hi;
                    if (pv) pv[v] = keep ? m : -1;
                    if (keep) {
#pragma unroll
                        for (int k = 0; k < C; ++k) acc[k] += (double)pts[(size_t)v * C + k];
                    }
                }
#pragma unroll
                for (int k = 0; k < C; ++k) {
#pragma unroll
                    for (int d = 16; d > 0; d >>= 1) acc[k] += __shfl_xor_sync(0xFFFFFFFFu, acc[k], d);
                }
                if (lane < C && m < a.capacity[sc]) {
                    double v = 0.0;
#pragma unroll
                    for (int k = 0; k < C; ++k) v = lane == k ? acc[k] : v;
                    const float mu = (float)(v / (double)g.cap);
                    a.mean[sc][(size_t)m * C + lane] = mu;
                    if (sc == 1 && a.bev) {
                        uint32_t r = g.ovf_cell[j];
                        const uint32_t x = r % g.dims[0]; r /= g.dims[0];
                        const uint32_t y = r % g.dims[1]; r /= g.dims[1];
                        const size_t plane = (size_t)g.dims[1] * g.dims[0];
                        a.bev[((size_t)r * C + lane) * plane + (size_t)y * g.dims[0] + x] = mu;
                    }
                }
            }
        }
        return;
    }
    // Voxel rows.  Occupied cells are first compacted into a shared list (their rows are
    // consecutive: the first one's rank plus the list position), then the list is worked off one
    // voxel per thread, so that accumulator reads and row writes are dense whatever the
    // occupancy pattern.
    __shared__ uint32_t s_cell[kThreads * 32];    // cell ids of one round; table mode: bit 31 = over the cap
    __shared__ int s_warp[kThreads / 32];
    __shared__ int s_first;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t t0 = a.ntiles_used[0], t1 = a.ntiles_used[1];
    const uint32_t nblk = gridDim.x - ovf_blocks;
    for (uint32_t v = blockIdx.x - ovf_blocks; v < t0 + t1; v += nblk) {
        const int sc = v >= t0 ? 1 : 0;
        const uint32_t tile = sc ? v - t0 : v;
        const ScaleDev& g = a.s[sc];
        if (!g.tile_flag[tile]) continue;
        const bool bitmap = g.mode == MODE_BITMAP;
        const int rounds = bitmap ? 4 : 2;        // 1024 words or 512 cells per tile, 256 per round
        for (int rnd = 0; rnd < rounds; ++rnd) {
            uint32_t bits = 0u, id0 = 0u;
            int rank = 0, k = 0;
            if (bitmap) {
                const uint32_t word = tile * (uint32_t)(4 * kThreads) + rnd * kThreads + threadIdx.x;
                uint2* pp = reinterpret_cast<uint2*>(g.store) + word;
                const uint2 pr = *pp;
                if (pr.x) *pp = make_uint2(0u, 0u);
                bits = pr.x; rank = (int)pr.y; id0 = word * 32u; k = __popc(bits);
            } else {
                const uint32_t cell = tile * (uint32_t)(2 * kThreads) + rnd * kThreads + threadIdx.x;
                uint4* pq = reinterpret_cast<uint4*>(g.store) + cell;
                const uint4 q = *pq;
                if (q.x) *pq = make_uint4(0u, 0u, 0u, 0u);
                bits = q.x ? 1u : 0u; rank = (int)q.y; k = (int)bits;
                id0 = cell | ((g.cap > 0 && (int)q.x > g.cap) ? 0x80000000u : 0u);
            }
            // Exclusive position of this thread's cells in the round's list.
            int inc = k;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                if (lane >= d) inc += y;
            }
            if (lane == 31) s_warp[warp] = inc;
            __syncthreads();
            int off = inc - k, total_k = 0;
#pragma unroll
            for (int w = 0; w < kThreads / 32; ++w) {
                const int c = s_warp[w];
                if (w < warp) off += c;
                total_k += c;
            }
            if (k > 0 && off == 0) s_first = rank;   // exactly one thread owns the round's first voxel
            if (bitmap) {
                while (bits) {
                    const int bit = __ffs(bits) - 1;
                    bits &= bits - 1;
                    s_cell[off++] = id0 + bit;
                }
            } else if (k) {
                s_cell[off] = id0;
            }
            __syncthreads();
            const int m0 = s_first;
            for (int i = threadIdx.x; i < total_k; i += kThreads) {
                const uint32_t c = s_cell[i];
                if (bitmap) write_voxel<C>(a, sc, g, m0 + i, c, false);
                else write_voxel<C>(a, sc, g, m0 + i, c & 0x7FFFFFFFu, (c >> 31) != 0u);
            }
            __syncthreads();
        }
    }
}

template <int C>
int run_voxelize(emc2_bridge* h, int B, int N, const float* d_points, int32_t* const d_coords[2],
                 int32_t* const d_counts[2], float* const d_mean[2], int32_t* const d_point_voxel[2],
                 const int32_t capacity[2], int32_t* d_num_voxels, float* d_bev, cudaStream_t st) {
    const long long total = (long long)B * N;
    const int ptiles = (int)((total + kBigTile - 1) / kBigTile);
    ScanArgs sa;
    AccumArgs aa;
    bool any_cap = false;
    for (int s = 0; s < 2; ++s) {
        sa.s[s] = h->scale[s];
        aa.s[s] = h->scale[s];
        const uint64_t cells = (uint64_t)B * h->scale[s].cells;
        const uint64_t per_tile = h->scale[s].mode == MODE_BITMAP ? kBitmapTileCells : kTableTileCells;
        sa.ntiles_used[s] = aa.ntiles_used[s] = (uint32_t)((cells + per_tile - 1) / per_tile);
        sa.capacity[s] = aa.capacity[s] = capacity[s];
        aa.coords[s] = d_coords[s];
        aa.counts[s] = d_counts[s];
        aa.mean[s] = d_mean[s];
        aa.point_voxel[s] = d_point_voxel ? d_point_voxel[s] : nullptr;
        any_cap = any_cap || h->scale[s].cap > 0;
    }
    sa.num_voxels = d_num_voxels;
    sa.status = h->d_status;
    sa.part = h->d_scan_part;
    aa.bev = d_bev;
    // Split the cooperative grid between the scales in proportion to their tile counts.
    const int G = h->scan_blocks;
    const double share = (double)sa.ntiles_used[0] / (double)((uint64_t)sa.ntiles_used[0] + sa.ntiles_used[1] + 1);
    sa.g0 = min(G - 1, max(1, (int)(share * G)));

    const size_t bev_n = d_bev ? (size_t)B * C * h->scale[1].dims[1] * h->scale[1].dims[0] : 0;
    const bool bev_vec = (bev_n & 3) == 0;
    if (bev_n && !bev_vec) cudaMemsetAsync(d_bev, 0, bev_n * sizeof(float), st);
    {
        // Also zeroes the BEV image; with no points it still runs for that.
        const int blocks = max(ptiles, (bev_n && bev_vec) ? 148 : 0);
        if (blocks > 0) {
            LaunchScope ls(h, K_VOX_MARK, st);
            vox_mark_kernel<C><<<blocks, kThreads, 0, st>>>(d_points, total, N, sa.s[0], sa.s[1],
                                                           bev_vec ? reinterpret_cast<float4*>(d_bev) : nullptr,
                                                           bev_vec ? bev_n >> 2 : 0);
        }
    }
    {
        LaunchScope ls(h, K_VOX_SCAN, st);
        void* args[] = {&sa};
        cudaError_t e = cudaLaunchCooperativeKernel((const void*)vox_scan_kernel, dim3(G), dim3(kThreads), args, 0, st);
        if (e != cudaSuccess) return check_cuda(h, e);
    }
    if (total > 0) {
        {
            LaunchScope ls(h, K_VOX_ACCUM, st);
            vox_accum_kernel<C><<<ptiles, kThreads, 0, st>>>(d_points, total, N, aa);
        }
        {
            // Which tiles hold voxels is only known on the device: a fixed grid strides over them.
            const int ovf_blocks = any_cap ? kOvfBlocks : 0;
            const uint32_t tiles = sa.ntiles_used[0] + sa.ntiles_used[1];
            const int vox_blocks = (int)min((uint32_t)(148 * 8), max(tiles, 1u));
            LaunchScope ls(h, K_VOX_FINALIZE, st);
            vox_finalize_kernel<C><<<ovf_blocks + vox_blocks, kThreads, 0, st>>>(d_points, total, aa, ovf_blocks);
        }
    }
    return check_cuda(h, cudaGetLastError());
}

}  // namespace

int voxel_scan_max_blocks() {
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, vox_scan_kernel, kThreads, 0) != cudaSuccess) return 0;
    int coop = 0;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) return 0;
    return sms * min(per_sm, 4);
}

int launch_voxelize(emc2_bridge* h, int B, int N, const float* d_points, int32_t* const d_coords[2],
                    int32_t* const d_counts[2], float* const d_mean[2], int32_t* const d_point_voxel[2],
                    const int32_t capacity[2], int32_t* d_num_voxels, float* d_bev, cudaStream_t st) {
    if (h->cfg.point_floats == 4)
        return run_voxelize<4>(h, B, N, d_points, d_coords, d_counts, d_mean, d_point_voxel, capacity,
                               d_num_voxels, d_bev, st);
    return run_voxelize<5>(h, B, N, d_points, d_coords, d_counts, d_mean, d_point_voxel, capacity,
                           d_num_voxels, d_bev, st);
}

}  // namespace emc2
