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
//   vox_count,    the rank scan, three launches: counts per 1 KB group of the store, prefix sums
//   vox_prefix,   of the per-CTA totals, then the exclusive prefix sums (the parallel prefix-sum
//   vox_rank      index search of Sec. 3.6) are written into the rank fields and the occupied
//                 cell ids listed in that order; accumulators are cleared and the bookkeeping of
//                 cells over the cap is laid out.
//   vox_accum     every point looks its rank up, writes point_voxel and adds itself to its
//                 voxels' accumulators with two fp32 vector reductions (offsets from the cell
//                 corner, the other channels, the count).
//                 Points of cells over the cap go to per-cell lists instead.
//   vox_finalize  a warp per 32 consecutive voxels: coordinates from the listed cell id, count,
//                 mean and BEV cell, with contiguous row traffic, and the store back to zero; in the same launch
//                 one warp per cell over the cap keeps the
//                 `cap` lowest point indices (keep-first-by-index) and sums them in fp64.
//
// Writes and reductions that land in one 32-byte sector are served one after another by the
// L2 (about 10 ns each on B200), so nothing here funnels many points into a shared flag or
// counter: the only contended words are the cells themselves.  The cost of a call follows the
// occupied groups, not the grid volume, except for one streaming read of the store.
#include "bridge_internal.cuh"

namespace emc2 {
namespace {

constexpr int kStatusCapacity = 1;
constexpr int kStatusDirtyStore = 8;   // the cell store held more than one call's points can set
constexpr int kPtsPerThread = 1;                      // points per thread of the two per-point passes (2 measured 1 - 3 % slower per step)
constexpr int kBigTile = kThreads * kPtsPerThread;    // points per CTA in the two per-point passes

// Where a point's cell sits in the unique list.
struct Slot {
    int m;      // row in the unique list, -1 if the point is outside the grid
    int j;      // rank among cells over the cap, -1 if the cell is not over it
};

__device__ __forceinline__ Slot slot_of(const ScaleDev& g, uint32_t cell, long long point) {
    Slot s;
    s.m = -1; s.j = -1;
    if (cell == 0xFFFFFFFFu) return s;
    if (g.design) {                               // hash / sort design: the row was computed per point
        s.m = g.point_rank[point];
        return s;
    }
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

// Exclusive scan of three counters across the warp; warp totals in tot[].
__device__ __forceinline__ void warp_excl_scan3(int v[3], int tot[3]) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        int x = v[k];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xFFFFFFFFu, x, d);
            if (lane >= d) x += y;
        }
        tot[k] = __shfl_sync(0xFFFFFFFFu, x, 31);
        v[k] = x - v[k];
    }
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
        mark_point(s0, s1, x, y, z, b0 + (i0 + t) / N);
    }
}

// ------------------------------------------------------------------ pass 2: ranks
struct ScanArgs {
    ScaleDev s[2];
    uint32_t ngroups_used[2];   // 1 KB groups covering this call's B frames
    int capacity[2];
    int32_t* num_voxels;
    int* status;
    int* cta_tot;               // [ctas0 + ctas1][3] voxels, cells over the cap and their points per CTA
    int* cta_base;              // same shape: exclusive prefix sums inside each scale
    int* unit_list;             // [ctas0 + ctas1] per scale: the CTAs of vox_count that found voxels, ascending
    int ctas0, ctas1;           // CTAs of vox_count / vox_rank serving scale 0 and scale 1
};

// One lane owns one 32-byte sector of the store: four {bits, rank} pairs or two cell records;
// a warp owns a 1 KB group.
struct Sector {
    uint4 a, b;
};

__device__ __forceinline__ Sector load_sector(const uint32_t* store, uint32_t group, int lane) {
    const uint4* p = reinterpret_cast<const uint4*>(store) + ((size_t)group * 32 + lane) * 2;
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

// Ranks and cell list of one group of a BITMAP store: a lane owns one 32-byte sector, i.e. four
// {bits, rank} words = 128 consecutive cells.  One warp scan of the lanes' popcounts places every
// word; each lane then lists its own cells (a handful in all but the densest groups) with plain
// stores that nothing waits for.  base0 = voxels before the group.
__device__ __forceinline__ void rank_group_bitmap(const ScaleDev& g, uint32_t grp, Sector x, int base0, int lane) {
    const uint32_t bw[4] = {x.a.x, x.a.z, x.b.x, x.b.z};
    const int c = __popc(bw[0]) + __popc(bw[1]) + __popc(bw[2]) + __popc(bw[3]);
    int inc = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= d) inc += y;
    }
    if (c == 0) return;
    int m = base0 + inc - c;
    const uint32_t word0 = (grp * 32u + lane) * 4u;
    uint32_t rk[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        rk[i] = (uint32_t)m;
        uint32_t bits = bw[i];
        while (bits) {
            const int bit = __ffs(bits) - 1;
            bits &= bits - 1;
            g.cell_list[m++] = (word0 + i) * 32u + bit;
        }
    }
    x.a.y = rk[0]; x.a.w = rk[1]; x.b.y = rk[2]; x.b.w = rk[3];
    uint4* p = reinterpret_cast<uint4*>(g.store) + ((size_t)grp * 32 + lane) * 2;
    p[0] = x.a;
    p[1] = x.b;
}

// Ranks, cell list and over-cap bookkeeping of one group of a TABLE store (two cell records per
// lane).  base[] = voxels, cells over the cap and points in such cells before the group.
__device__ __forceinline__ void rank_group_table(const ScaleDev& g, uint32_t grp, Sector x, const int base[3], int lane) {
    int run[3] = {0, 0, 0}, gtot[3];
    sector_stats(g, x, run);
    const bool mine = run[0] > 0;
    warp_excl_scan3(run, gtot);                   // run[] = exclusive offsets inside the group
    if (!mine) return;
    int m = base[0] + run[0];
    int j = base[1] + run[1], off = base[2] + run[2];
    const uint32_t cell0 = (grp * 32u + lane) * 2u;
    x.a.y = (uint32_t)m; x.a.z = (uint32_t)j;
    const int n0 = (int)x.a.x, n1 = (int)x.b.x;
    const bool o0 = g.cap > 0 && n0 > g.cap, o1 = g.cap > 0 && n1 > g.cap;
    if (o0) {
        g.ovf_vox[j] = m; g.ovf_off[j] = off; g.ovf_cell[j] = cell0; g.ovf_cursor[(size_t)j * kCursorStride] = 0;
        j += 1; off += n0;
    }
    if (n0 > 0) g.cell_list[m++] = cell0 | (o0 ? 0x80000000u : 0u);
    x.b.y = (uint32_t)m; x.b.z = (uint32_t)j;
    if (o1) {
        g.ovf_vox[j] = m; g.ovf_off[j] = off; g.ovf_cell[j] = cell0 + 1u; g.ovf_cursor[(size_t)j * kCursorStride] = 0;
    }
    if (n1 > 0) g.cell_list[m] = (cell0 + 1u) | (o1 ? 0x80000000u : 0u);
    uint4* p = reinterpret_cast<uint4*>(g.store) + ((size_t)grp * 32 + lane) * 2;
    p[0] = x.a;
    p[1] = x.b;
}

// The rank scan is three plain launches, each a few memory round trips deep, so that it keeps its
// pace when it runs beside kernels that saturate the memory system (a deep chain of dependent loads
// stretches with the latency of every hop).  A CTA owns 32 consecutive groups of one scale, a warp
// four of them.
//   vox_count   streams the store once: per-group counts into group_info, per-CTA totals.
//   vox_prefix  one CTA per scale: exclusive prefix sums of the CTA totals, the scale's totals, the
//               number of voxels and the capacity / consistency checks.
//   vox_rank    a warp turns its CTA's 32 group counts into group bases with one warp scan, loads
//               only its occupied groups (all at once), writes their ranks and lists their cells in
//               rank order: the parallel prefix-sum index search of Sec. 3.6.  Also clears the
//               accumulators of the voxels found.
constexpr int kGroupsPerWarp = 4;
constexpr int kGroupsPerCta = kGroupsPerWarp * (kThreads / 32);
static_assert(kGroupsPerCta == 32, "vox_rank_kernel scans one group count per lane");

__global__ void __launch_bounds__(kThreads) vox_count_kernel(ScanArgs a) {
    constexpr int kWarps = kThreads / 32;
    __shared__ int wtot[kWarps][3];
    const int sc = (int)blockIdx.x >= a.ctas0 ? 1 : 0;
    const uint32_t cta = blockIdx.x - (sc ? a.ctas0 : 0);
    const ScaleDev& g = a.s[sc];
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const uint32_t ng = a.ngroups_used[sc];
    const uint32_t g0 = cta * kGroupsPerCta + warp * kGroupsPerWarp;
    Sector x[kGroupsPerWarp];
#pragma unroll
    for (int u = 0; u < kGroupsPerWarp; ++u) {
        x[u].a = x[u].b = make_uint4(0u, 0u, 0u, 0u);
        if (g0 + u < ng) {
            const uint4* p = reinterpret_cast<const uint4*>(g.store) + ((size_t)(g0 + u) * 32 + lane) * 2;
            x[u].a = __ldcs(p);                   // streaming: most of the store is empty, keep it out of L2
            x[u].b = __ldcs(p + 1);
        }
    }
    int carry[3] = {0, 0, 0};
#pragma unroll
    for (int u = 0; u < kGroupsPerWarp; ++u) {
        int s[3] = {0, 0, 0};
        sector_stats(g, x[u], s);
#pragma unroll
        for (int k = 0; k < 3; ++k) s[k] = warp_sum(s[k]);
        if (lane == 0 && g0 + u < ng) g.group_info[g0 + u] = make_int4(s[0], s[1], s[2], 0);
#pragma unroll
        for (int k = 0; k < 3; ++k) carry[k] += s[k];
    }
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < 3; ++k) wtot[warp][k] = carry[k];
    }
    __syncthreads();
    if (t < 3) {
        int v = 0;
        for (int w = 0; w < kWarps; ++w) v += wtot[w][t];
        a.cta_tot[(size_t)blockIdx.x * 3 + t] = v;
    }
}

constexpr int kPrefixThreads = 1024;

// grid = 2: CTA sc scans the CTA totals of scale sc.  It also lists the CTAs that found any voxel
// (most of a fine grid is empty space), so that the ranking pass only visits those.
__global__ void __launch_bounds__(kPrefixThreads) vox_prefix_kernel(ScanArgs a) {
    constexpr int kWarps = kPrefixThreads / 32;
    __shared__ int wsum[4][kWarps];
    __shared__ int tot[4];
    const int sc = blockIdx.x;
    const ScaleDev& g = a.s[sc];
    if (g.design) return;                         // ranked by another design: its totals stand
    const int first = sc ? a.ctas0 : 0, n = sc ? a.ctas1 : a.ctas0;
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int per = (n + kPrefixThreads - 1) / kPrefixThreads;
    const int lo = min(n, t * per), hi = min(n, lo + per);
    const int* src = a.cta_tot + (size_t)first * 3;
    int* dst = a.cta_base + (size_t)first * 3;
    int run[4] = {0, 0, 0, 0};                    // voxels, cells over the cap, their points, CTAs with voxels
    for (int i = lo; i < hi; ++i) {
#pragma unroll
        for (int k = 0; k < 3; ++k) run[k] += src[(size_t)i * 3 + k];
        run[3] += src[(size_t)i * 3] > 0;
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {                 // run[] becomes exclusive inside the warp
        int x = run[k];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xFFFFFFFFu, x, d);
            if (lane >= d) x += y;
        }
        if (lane == 31) wsum[k][warp] = x;
        run[k] = x - run[k];
    }
    __syncthreads();
    if (warp < 4) {                               // warp k scans the warp totals of counter k
        int x = wsum[warp][lane];
        const int v = x;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xFFFFFFFFu, x, d);
            if (lane >= d) x += y;
        }
        wsum[warp][lane] = x - v;
        if (lane == 31) tot[warp] = x;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) run[k] += wsum[k][warp];
    for (int i = lo; i < hi; ++i) {
#pragma unroll
        for (int k = 0; k < 3; ++k) dst[(size_t)i * 3 + k] = run[k];
        const int v0 = src[(size_t)i * 3];
        if (v0 > 0) a.unit_list[first + run[3]++] = i;
#pragma unroll
        for (int k = 0; k < 3; ++k) run[k] += src[(size_t)i * 3 + k];
    }
    if (t == 0) {
        // More voxels, cells over the cap or points in them than a call's points allow: the store was
        // not all zero when the call began (two calls on one handle at once).  Nothing is ranked or
        // listed then; the scale reports no voxels and the handle's status becomes an internal error.
        const bool dirty = (uint32_t)tot[0] > g.max_list || (uint32_t)tot[1] > g.max_ovf || (uint32_t)tot[2] > g.max_list;
        g.totals[0] = dirty ? 0 : tot[0]; g.totals[1] = dirty ? 0 : tot[1]; g.totals[2] = dirty ? 0 : tot[2];
        g.totals[3] = dirty ? 0 : tot[3];         // CTAs the ranking pass has to visit
        a.num_voxels[sc] = dirty ? 0 : tot[0];
        if (dirty) atomicOr(a.status, kStatusDirtyStore);
        else if (tot[0] > a.capacity[sc]) atomicOr(a.status, kStatusCapacity);
    }
}

// A fixed grid: every CTA first clears its share of the accumulators of the voxels found (two
// 16-byte halves per voxel), then takes the listed units (32 groups of one scale) in turn.
__global__ void __launch_bounds__(kThreads, 5) vox_rank_kernel(ScanArgs a) {
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int n0 = a.s[0].totals[3], n1 = a.s[1].totals[3];
    const int v0 = a.s[0].totals[0], v1 = a.s[1].totals[0];
    {
        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        const size_t c0 = 2 * (size_t)v0, c1 = 2 * (size_t)v1;
        for (size_t i = (size_t)blockIdx.x * kThreads + t; i < c0 + c1; i += (size_t)gridDim.x * kThreads) {
            if (i < c0) a.s[0].acc[i] = z; else a.s[1].acc[i - c0] = z;
        }
    }
    for (int u = blockIdx.x; u < n0 + n1; u += gridDim.x) {
        const int sc = u >= n0 ? 1 : 0;
        const ScaleDev& g = a.s[sc];
        const int first = sc ? a.ctas0 : 0;
        const uint32_t cta = (uint32_t)a.unit_list[first + (sc ? u - n0 : u)];
        const uint32_t ng = a.ngroups_used[sc];
        const uint32_t gc = cta * kGroupsPerCta;
        int pre[3] = {0, 0, 0}, ctot[3];
        if (gc + lane < ng) {
            const int4 info = g.group_info[gc + lane];
            pre[0] = info.x; pre[1] = info.y; pre[2] = info.z;
        }
        int base[3];
#pragma unroll
        for (int k = 0; k < 3; ++k) base[k] = a.cta_base[(size_t)(first + cta) * 3 + k];
        const unsigned occupied = __ballot_sync(0xFFFFFFFFu, pre[0] > 0);
        const bool bitmap = g.mode == MODE_BITMAP;
        // The unit's occupied groups are dealt to the warps round-robin (a unit in open space has a few,
        // one on the ground plane all 32); a warp requests all of its groups before it ranks any.
        const int nocc = __popc(occupied);
        int gidx[kGroupsPerWarp];
        Sector x[kGroupsPerWarp];
#pragma unroll
        for (int i = 0; i < kGroupsPerWarp; ++i) {
            const int k = warp + i * (kThreads / 32);
            gidx[i] = k < nocc ? (int)__fns(occupied, 0, k + 1) : -1;
            if (gidx[i] >= 0) x[i] = load_sector(g.store, gc + gidx[i], lane);
        }
        warp_excl_scan3(pre, ctot);               // pre[] = what the unit's groups before this lane's group hold
#pragma unroll
        for (int i = 0; i < kGroupsPerWarp; ++i) {
            if (gidx[i] < 0) break;
            int gb[3];
#pragma unroll
            for (int k = 0; k < 3; ++k) gb[k] = base[k] + __shfl_sync(0xFFFFFFFFu, pre[k], gidx[i]);
            if (bitmap) rank_group_bitmap(g, gc + gidx[i], x[i], gb[0], lane);
            else rank_group_table(g, gc + gidx[i], x[i], gb, lane);
        }
    }
}

// ------------------------------------------------------------------ pass 3: accumulate
struct AccumArgs {
    ScaleDev s[2];
    uint32_t ngroups_used[2];
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
    // All rank lookups first, so that a thread has its loads in flight together.
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
            slot[sc][i] = slot_of(g, cell, g0 + t);
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
                if ((uint32_t)s.j < g.max_ovf) {      // always, unless the store was dirty
                    const int tk = atomicAdd(&g.ovf_cursor[(size_t)s.j * kCursorStride], 1);
                    const uint32_t pos = (uint32_t)(g.ovf_off[s.j] + tk);
                    if (pos < g.max_list) g.ovf_list[pos] = (int)(g0 + t);
                }
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

// ------------------------------------------------------------------ per-voxel cap on a bitmap scale
// A bitmap store keeps no per-cell point count, so a voxel over its cap is only known once the points
// are accumulated.  Two small passes then build what the table path gets from the rank scan:
//   vox_over_find   a thread per voxel row: count > cap -> the voxel takes the next place j among the
//                   over-cap voxels and the next `count` slots of the index list (warp-aggregated
//                   tickets), and remembers j + 1 in the spare word of its accumulator;
//   vox_over_fill   a thread per point: if its voxel is over the cap, the point's index goes into the
//                   voxel's list.
// vox_finalize then keeps the `cap` lowest indices of every list exactly as for a table scale.
__global__ void __launch_bounds__(kThreads) vox_over_find_kernel(AccumArgs a, int sc) {
    const ScaleDev& g = a.s[sc];
    const int lane = threadIdx.x & 31;
    const int M = min(g.totals[0], a.capacity[sc]);
    for (int m0 = (blockIdx.x * kThreads + threadIdx.x) & ~31; m0 < M; m0 += gridDim.x * kThreads) {
        const int m = m0 + lane;
        const int n = m < M ? (int)g.acc[2 * (size_t)m + 1].y : 0;
        const bool over = n > g.cap;
        const unsigned who = __ballot_sync(0xFFFFFFFFu, over);
        if (!who) continue;
        int inc = over ? n : 0;                   // inclusive scan of the over-cap counts
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
            if (lane >= d) inc += y;
        }
        int j0 = 0, off0 = 0;
        if (lane == 31) {
            j0 = atomicAdd(&g.totals[1], __popc(who));
            off0 = atomicAdd(&g.totals[2], inc);
        }
        j0 = __shfl_sync(0xFFFFFFFFu, j0, 31);
        off0 = __shfl_sync(0xFFFFFFFFu, off0, 31);
        if (!over) continue;
        const int j = j0 + __popc(who & ((1u << lane) - 1u));
        const int off = off0 + inc - n;
        if ((uint32_t)j >= g.max_ovf || (uint32_t)(off + n) > g.max_list) continue;   // cannot happen with this batch's counts
        g.ovf_vox[j] = m; g.ovf_off[j] = off; g.ovf_cell[j] = g.cell_list[m];
        g.ovf_cursor[(size_t)j * kCursorStride] = 0;
        reinterpret_cast<uint32_t*>(g.acc + 2 * (size_t)m + 1)[2] = (uint32_t)j + 1u;
    }
}

template <int C>
__global__ void __launch_bounds__(kThreads)
vox_over_fill_kernel(const float* __restrict__ pts, long long total, int N, AccumArgs a, int sc) {
    const ScaleDev& g = a.s[sc];
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < total; i += (long long)gridDim.x * kThreads) {
        const float* p = pts + i * C;
        const Slot s = slot_of(g, cell_of(g, p[0], p[1], p[2], (int)(i / N)), i);
        if (s.m < 0 || s.m >= a.capacity[sc]) continue;
        const uint32_t tag = reinterpret_cast<const uint32_t*>(g.acc + 2 * (size_t)s.m + 1)[2];
        if (tag == 0u || tag > g.max_ovf) continue;
        const int j = (int)tag - 1;
        const int tk = atomicAdd(&g.ovf_cursor[(size_t)j * kCursorStride], 1);
        const uint32_t pos = (uint32_t)(g.ovf_off[j] + tk);
        if (pos < g.max_list) g.ovf_list[pos] = (int)i;
    }
}

// ------------------------------------------------------------------ pass 4: rows, BEV, cleanup
// Writes the output rows of n <= 32 voxels with consecutive rows mb, mb+1, ..., one per lane;
// lane i holds the cell-list entry of row mb + i; `stage` is 1 KB of the warp's own shared memory.  Accumulators are read and mean rows written as
// contiguous blocks through shared memory, so the warp issues full-sector requests only.
template <int C>
__device__ __forceinline__ void write_batch(const AccumArgs& a, int sc, int mb, int n, uint32_t entry,
                                            float4* stage) {
    const ScaleDev& g = a.s[sc];
    const int lane = threadIdx.x & 31;
    n = min(n, a.capacity[sc] - mb);              // rows past the caller's capacity are not written
    if (n <= 0) return;
    const float4* src = g.acc + 2 * (size_t)mb;
    if (lane < 2 * n) stage[lane] = src[lane];
    if (lane + 32 < 2 * n) stage[lane + 32] = src[lane + 32];
    __syncwarp();
    const float4 a0 = stage[2 * lane], a1 = stage[2 * lane + 1];
    __syncwarp();
    const bool active = lane < n;
    const bool table = g.mode == MODE_TABLE;
    const uint32_t cell = table ? (entry & 0x7FFFFFFFu) : entry;
    // Over the cap: a table store flags the cell in its list entry; a bitmap store has no per-cell count,
    // there vox_over_find_kernel left the voxel's place among the over-cap voxels (+ 1) in a spare word.
    const bool over = active && ((table && (entry >> 31) != 0u) || __float_as_uint(a1.z) != 0u);
    uint32_t r = cell, x, y, z;
    g.div[0].divmod(r, r, x);
    g.div[1].divmod(r, r, y);
    g.div[2].divmod(r, r, z);
    const int cnt = over ? g.cap : (int)a1.y;
    // Offsets are below one cell size, so fp32 keeps the mean to a few 1e-7 of that size.
    const float inv = __frcp_rn((float)cnt);
    float mu[C];
    mu[0] = __fadd_rn(cell_corner(g.mn[0], g.vs[0], (int)x), a0.x * inv);
    mu[1] = __fadd_rn(cell_corner(g.mn[1], g.vs[1], (int)y), a0.y * inv);
    mu[2] = __fadd_rn(cell_corner(g.mn[2], g.vs[2], (int)z), a0.z * inv);
    mu[3] = __fdiv_rn(a0.w, (float)cnt);
    if (C > 4) mu[4] = __fdiv_rn(a1.x, (float)cnt);
    if (active) {
        reinterpret_cast<int4*>(a.coords[sc])[mb + lane] = make_int4((int)r, (int)z, (int)y, (int)x);
        a.counts[sc][mb + lane] = cnt;
    }
    // Mean rows: the n * C floats of rows mb .. mb+n-1 are contiguous.  The row of a cell over the
    // cap is written by that cell's own warp, so a batch holding one writes its rows one by one.
    float* rows = a.mean[sc] + (size_t)mb * C;
    if (!__any_sync(0xFFFFFFFFu, over)) {
        float* st = reinterpret_cast<float*>(stage);
#pragma unroll
        for (int k = 0; k < C; ++k) st[lane * C + k] = mu[k];
        __syncwarp();
        for (int i = lane; i < n * C; i += 32) rows[i] = st[i];
        __syncwarp();
    } else if (active && !over) {
#pragma unroll
        for (int k = 0; k < C; ++k) rows[lane * C + k] = mu[k];
    }
    if (sc == 1 && a.bev && active && !over) {
        const size_t plane = (size_t)g.dims[1] * g.dims[0];
        float* dst = a.bev + (size_t)r * C * plane + (size_t)y * g.dims[0] + x;
#pragma unroll
        for (int k = 0; k < C; ++k) dst[(size_t)k * plane] = mu[k];
    }
}

// CTAs [0, ovf_blocks) serve cells over the cap, one warp per cell: the `cap` lowest point
// indices are kept (keep-first-by-index), summed in fp64 and written as the voxel's mean; all of
// the cell's points get their point_voxel entry.  The other CTAs write the voxel rows.
template <int C>
__global__ void __launch_bounds__(kThreads)
vox_finalize_kernel(const float* __restrict__ pts, long long total, AccumArgs a, int ovf_blocks) {
    constexpr int kWarps = kThreads / 32;
    const int lane = threadIdx.x & 31;
    if ((int)blockIdx.x < ovf_blocks) {
        const int warp = (blockIdx.x * kThreads + threadIdx.x) >> 5;
        const int nwarps = ovf_blocks * kWarps;
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
                        uint32_t r = g.ovf_cell[j], x, y;
                        g.div[0].divmod(r, r, x);
                        g.div[1].divmod(r, r, y);
                        const size_t plane = (size_t)g.dims[1] * g.dims[0];
                        a.bev[((size_t)r * C + lane) * plane + (size_t)y * g.dims[0] + x] = mu;
                    }
                }
            }
        }
        return;
    }
    // Voxel rows: a warp takes 32 consecutive rows of one scale at a time, reads their cell ids
    // from the list the rank scan wrote, writes the rows and puts the cells' store words back to
    // zero (whole 32-byte sectors of a bitmap store: a partial write would first fetch the sector).
    // Every warp has its own batch, so the batches' memory latencies overlap.
    __shared__ float4 s_stage[kWarps][64];
    float4* stage = s_stage[threadIdx.x >> 5];
    const int tot0 = a.s[0].totals[0], tot1 = a.s[1].totals[0];
    const int nb0 = (tot0 + 31) >> 5, nb1 = (tot1 + 31) >> 5;
    const int nwarps = ((int)gridDim.x - ovf_blocks) * kWarps;
    for (int v = ((int)blockIdx.x - ovf_blocks) * kWarps + (threadIdx.x >> 5); v < nb0 + nb1; v += nwarps) {
        const int sc = v >= nb0 ? 1 : 0;
        const int mb = (sc ? v - nb0 : v) << 5;
        const ScaleDev& g = a.s[sc];
        const int n = min(32, (sc ? tot1 : tot0) - mb);
        const uint32_t entry = lane < n ? g.cell_list[mb + lane] : 0u;
        if (lane < n && !g.design) {
            if (g.mode == MODE_BITMAP) {
                uint4* sp = reinterpret_cast<uint4*>(g.store + 8 * (size_t)(entry >> 7));
                sp[0] = make_uint4(0u, 0u, 0u, 0u);
                sp[1] = make_uint4(0u, 0u, 0u, 0u);
            } else {
                *reinterpret_cast<uint4*>(g.store + 4 * (size_t)(entry & 0x7FFFFFFFu)) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        write_batch<C>(a, sc, mb, n, entry, stage);
    }
}

template <int C>
int run_voxelize(emc2_bridge* h, int B, int N, const float* d_points, int32_t* const d_coords[2],
                 int32_t* const d_counts[2], float* const d_mean[2], int32_t* const d_point_voxel[2],
                 const int32_t capacity[2], int32_t* d_num_voxels, float* d_bev, cudaStream_t st, bool marked) {
    const long long total = (long long)B * N;
    const int ptiles = (int)((total + kBigTile - 1) / kBigTile);
    ScanArgs sa;
    AccumArgs aa;
    bool any_cap = false;
    for (int s = 0; s < 2; ++s) {
        sa.s[s] = h->scale[s];
        // A scale deduplicated by the hash or sort design has no store to scan; its voxel list is a plain
        // list of cell ids, which the later passes treat like a bitmap scale's.
        if (sa.s[s].design) sa.s[s].mode = MODE_BITMAP;
        aa.s[s] = sa.s[s];
        const uint64_t cells = sa.s[s].design ? 0 : (uint64_t)B * h->scale[s].cells;
        const uint64_t per_group = h->scale[s].mode == MODE_BITMAP ? kBitmapGroupCells : kTableGroupCells;
        sa.ngroups_used[s] = aa.ngroups_used[s] = (uint32_t)((cells + per_group - 1) / per_group);
        sa.capacity[s] = aa.capacity[s] = capacity[s];
        aa.coords[s] = d_coords[s];
        aa.counts[s] = d_counts[s];
        aa.mean[s] = d_mean[s];
        aa.point_voxel[s] = d_point_voxel ? d_point_voxel[s] : nullptr;
        any_cap = any_cap || h->scale[s].cap > 0;
    }
    sa.num_voxels = d_num_voxels;
    sa.status = h->d_status;
    sa.cta_tot = h->d_scan_tot;
    sa.cta_base = h->d_scan_base;
    sa.unit_list = h->d_scan_units;
    sa.ctas0 = (int)((sa.ngroups_used[0] + kGroupsPerCta - 1) / kGroupsPerCta);
    sa.ctas1 = (int)((sa.ngroups_used[1] + kGroupsPerCta - 1) / kGroupsPerCta);
    aa.bev = d_bev;

    const size_t bev_n = d_bev ? (size_t)B * C * h->scale[1].dims[1] * h->scale[1].dims[0] : 0;
    const bool bev_vec = (bev_n & 3) == 0;
    if (!marked && bev_n && !bev_vec) cudaMemsetAsync(d_bev, 0, bev_n * sizeof(float), st);
    if (!marked) {
        // Also zeroes the BEV image; with no points it still runs for that.
        const int blocks = max(ptiles, (bev_n && bev_vec) ? h->num_sms : 0);
        if (blocks > 0) {
            LaunchScope ls(h, K_VOX_MARK, st);
            vox_mark_kernel<C><<<blocks, kThreads, 0, st>>>(d_points, total, N, sa.s[0], sa.s[1],
                                                           bev_vec ? reinterpret_cast<float4*>(d_bev) : nullptr,
                                                           bev_vec ? bev_n >> 2 : 0);
        }
    }
    for (int s = 0; s < 2; ++s) {
        if (!h->scale[s].design) continue;
        const int rc = launch_dedup_arm(h, s, h->scale[s].design, B, N, d_points, capacity[s], d_num_voxels, st);
        if (rc != EMC2_OK) return rc;
    }
    if (sa.ctas0 + sa.ctas1 > 0) {
        LaunchScope ls(h, K_VOX_COUNT, st);
        vox_count_kernel<<<sa.ctas0 + sa.ctas1, kThreads, 0, st>>>(sa);
    }
    {
        LaunchScope ls(h, K_VOX_PREFIX, st);      // with no frames it still reports zero voxels
        vox_prefix_kernel<<<2, kPrefixThreads, 0, st>>>(sa);
    }
    if (sa.ctas0 + sa.ctas1 > 0) {
        LaunchScope ls(h, K_VOX_RANK, st);
        vox_rank_kernel<<<min(sa.ctas0 + sa.ctas1, 5 * h->num_sms), kThreads, 0, st>>>(sa);
    }
    if (total > 0) {
        LaunchScope ls(h, K_VOX_ACCUM, st);
        vox_accum_kernel<C><<<ptiles, kThreads, 0, st>>>(d_points, total, N, aa);
    }
    for (int s = 0; s < 2 && total > 0; ++s) {
        if (aa.s[s].mode != MODE_BITMAP || h->scale[s].cap <= 0) continue;
        {
            LaunchScope ls(h, K_VOX_OVER_FIND, st);
            vox_over_find_kernel<<<4 * h->num_sms, kThreads, 0, st>>>(aa, s);
        }
        {
            LaunchScope ls(h, K_VOX_OVER_FILL, st);
            vox_over_fill_kernel<C><<<(int)min((long long)8 * h->num_sms, (total + kThreads - 1) / kThreads), kThreads, 0, st>>>(
                d_points, total, N, aa, s);
        }
    }
    if (total > 0) {
        // The number of voxels is only known on the device: a fixed grid strides over them.
        const int ovf_blocks = any_cap ? 2 * h->num_sms : 0;    // CTAs that serve cells over the cap
        const int vox_blocks = (int)min((long long)h->num_sms * 8, (2 * total + 32 * 8 - 1) / (32 * 8) + 1);
        LaunchScope ls(h, K_VOX_FINALIZE, st);
        vox_finalize_kernel<C><<<ovf_blocks + vox_blocks, kThreads, 0, st>>>(d_points, total, aa, ovf_blocks);
    }
    return check_cuda(h, cudaGetLastError());
}

}  // namespace

int launch_voxelize(emc2_bridge* h, int B, int N, const float* d_points, int32_t* const d_coords[2],
                    int32_t* const d_counts[2], float* const d_mean[2], int32_t* const d_point_voxel[2],
                    const int32_t capacity[2], int32_t* d_num_voxels, float* d_bev, cudaStream_t st, bool marked) {
    if (h->cfg.point_floats == 4)
        return run_voxelize<4>(h, B, N, d_points, d_coords, d_counts, d_mean, d_point_voxel, capacity,
                               d_num_voxels, d_bev, st, marked);
    return run_voxelize<5>(h, B, N, d_points, d_coords, d_counts, d_mean, d_point_voxel, capacity,
                           d_num_voxels, d_bev, st, marked);
}

}  // namespace emc2
