// Stage 1 of the bridge: two-scale voxelization, dedup in canonical order, per-voxel counts
// and means, BEV scatter (Sec. 3.1 preprocessing; BEV for the 2D expert of Sec. 3.3).
//
// Dedup is direct-addressed, with no sort: every cell of the batch owns one bit (large grids)
// or one 32-bit counter (grids small enough for a count table).  The store is cut into
// 32-byte chunks (one L2 sector: 256 bitmap cells or 8 counters); a summary bitmap holds one
// bit per chunk.  Points mark their cell with one atomic; a prefix sum over the occupied
// chunks (the parallel prefix-sum index search of Sec. 3.6) then gives every occupied cell its
// rank in ascending (b, z, y, x) order, which is the canonical voxel order.  A second pass
// over the points looks the rank up (one sector load plus popcounts) and accumulates: the
// first point to reach a voxel stores its values straight into the output row, later points
// add into fp64 scratch sums.  A per-voxel pass writes coordinates, counts, means and the BEV
// image and puts every scratch word it used back to zero, so the cost of a call follows the
// occupied cells, not the grid volume.
#include "bridge_internal.cuh"

namespace emc2 {
namespace {

constexpr int kStatusCapacity = 1;
constexpr int kPtsPerThread = 4;                      // independent points per thread (memory-level parallelism)
constexpr int kBigTile = kThreads * kPtsPerThread;    // points per CTA in the two per-point passes

// ------------------------------------------------------------------ block-level helpers
// Exclusive scan of three counters across the CTA; returns CTA totals in tot[].
__device__ __forceinline__ void block_excl_scan3(int v[3], int tot[3], int (*sm)[3]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    int inc[3];
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        int x = v[k];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            int y = __shfl_up_sync(0xFFFFFFFFu, x, d);
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
                int y = __shfl_up_sync(0xFFFFFFFFu, x, d);
                if (lane >= d) x += y;
            }
            if (lane < nwarp) sm[lane][k] = x;   // inclusive over warps
        }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        int wbase = warp ? sm[warp - 1][k] : 0;
        tot[k] = sm[nwarp - 1][k];
        v[k] = wbase + inc[k] - v[k];
    }
    __syncthreads();
}

struct Chunk {
    uint32_t w[8];
};

__device__ __forceinline__ Chunk load_chunk(const uint32_t* store, uint32_t chunk) {
    const uint4* p = reinterpret_cast<const uint4*>(store + (size_t)chunk * 8);
    uint4 a = p[0], b = p[1];
    Chunk c;
    c.w[0] = a.x; c.w[1] = a.y; c.w[2] = a.z; c.w[3] = a.w;
    c.w[4] = b.x; c.w[5] = b.y; c.w[6] = b.z; c.w[7] = b.w;
    return c;
}

// Occupied cells, overflowing cells and points in overflowing cells of one chunk.
__device__ __forceinline__ void chunk_stats(const ScaleDev& g, const Chunk& c, int s[3]) {
    if (g.mode == MODE_BITMAP) {
#pragma unroll
        for (int i = 0; i < 8; ++i) s[0] += __popc(c.w[i]);
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            int n = (int)c.w[i];
            s[0] += n > 0;
            if (g.cap > 0 && n > g.cap) { s[1] += 1; s[2] += n; }
        }
    }
}

// Where a point's cell sits in the unique list.
struct Slot {
    int m;      // row in the unique list, -1 if the point is outside the grid
    int n;      // points in the cell (count table only)
    int j;      // rank among cells that exceed the cap, -1 if the cell does not
};

__device__ __forceinline__ Slot slot_of(const ScaleDev& g, uint32_t cell) {
    Slot s;
    s.m = -1; s.n = 0; s.j = -1;
    if (cell == 0xFFFFFFFFu) return s;
    if (g.mode == MODE_BITMAP) {
        const uint32_t chunk = cell >> 8, w = (cell >> 5) & 7u, bit = cell & 31u;
        const Chunk c = load_chunk(g.store, chunk);
        uint32_t r = g.chunk_prefix[chunk];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            uint32_t mask = i < (int)w ? 0xFFFFFFFFu : (i == (int)w ? ((1u << bit) - 1u) : 0u);
            r += __popc(c.w[i] & mask);
        }
        s.m = (int)r;
    } else {
        const uint32_t chunk = cell >> 3, w = cell & 7u;
        const Chunk c = load_chunk(g.store, chunk);
        uint32_t r = g.chunk_prefix[chunk];
        int before_ovf = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            r += (i < (int)w && c.w[i] != 0u) ? 1u : 0u;
            before_ovf += (i < (int)w && g.cap > 0 && (int)c.w[i] > g.cap) ? 1 : 0;
        }
        int n = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) n = i == (int)w ? (int)c.w[i] : n;   // no dynamic register indexing
        s.m = (int)r;
        s.n = n;
        if (g.cap > 0 && n > g.cap) s.j = (int)g.chunk_ovf[chunk] + before_ovf;
    }
    return s;
}

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
    uint32_t cell[2][kPtsPerThread];
#pragma unroll
    for (int i = 0; i < kPtsPerThread; ++i) {
        const int t = threadIdx.x + i * kThreads;
        cell[0][i] = cell[1][i] = 0xFFFFFFFFu;
        if (t < npts) {
            const float x = sp[t * C], y = sp[t * C + 1], z = sp[t * C + 2];
            const int b = (int)((g0 + t) / N);
            cell[0][i] = cell_of(s0, x, y, z, b);
            cell[1][i] = cell_of(s1, x, y, z, b);
        }
    }
    // All marking atomics are issued before any result is consumed.
    uint32_t old[2][kPtsPerThread];
#pragma unroll
    for (int sc = 0; sc < 2; ++sc) {
        const ScaleDev& g = sc ? s1 : s0;
#pragma unroll
        for (int i = 0; i < kPtsPerThread; ++i) {
            const uint32_t c = cell[sc][i];
            old[sc][i] = 1u;
            if (c != 0xFFFFFFFFu)
                old[sc][i] = g.mode == MODE_BITMAP ? atomicOr(&g.store[c >> 5], 1u << (c & 31u))
                                                   : atomicAdd(&g.store[c], 1u);
        }
    }
#pragma unroll
    for (int sc = 0; sc < 2; ++sc) {
        const ScaleDev& g = sc ? s1 : s0;
        const int shift = g.mode == MODE_BITMAP ? 8 : 3;
#pragma unroll
        for (int i = 0; i < kPtsPerThread; ++i) {
            if (old[sc][i] == 0u) {              // first touch of a word / cell: flag its chunk
                const uint32_t chunk = cell[sc][i] >> shift;
                atomicOr(&g.summary[chunk >> 5], 1u << (chunk & 31u));
            }
        }
    }
}

// ------------------------------------------------------------------ pass 2: ranks
struct ScanArgs {
    ScaleDev s[2];
    uint32_t nchunks_used[2];   // chunks covering this call's B frames
    int capacity[2];
    int32_t* num_voxels;
    int* status;
};

__device__ __forceinline__ bool chunk_flagged(const ScaleDev& g, uint32_t chunk, uint32_t nchunks) {
    return chunk < nchunks && ((g.summary[chunk >> 5] >> (chunk & 31u)) & 1u);
}

// One thread per chunk; per-CTA totals of (voxels, overflowing voxels, overflowing points).
__global__ void __launch_bounds__(kThreads) vox_reduce_kernel(ScanArgs a) {
    __shared__ int sm[kThreads / 32][3];
    const int sc = blockIdx.y;
    const ScaleDev& g = a.s[sc];
    const uint32_t nblk = (a.nchunks_used[sc] + kThreads - 1) / kThreads;
    if (blockIdx.x >= nblk) return;
    const uint32_t chunk = blockIdx.x * kThreads + threadIdx.x;
    int s[3] = {0, 0, 0};
    if (chunk_flagged(g, chunk, a.nchunks_used[sc])) chunk_stats(g, load_chunk(g.store, chunk), s);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        int v = warp_sum(s[k]);
        if (lane == 0) sm[warp][k] = v;
    }
    __syncthreads();
    if (threadIdx.x < 3) {
        int v = 0;
        for (int w = 0; w < kThreads / 32; ++w) v += sm[w][threadIdx.x];
        g.blk_sums[blockIdx.x * 3 + threadIdx.x] = v;
    }
}

// One CTA per scale: exclusive scan of the per-CTA sums (each thread owns a run of
// consecutive entries, so one CTA-wide scan covers 1024 * run entries); totals, capacity check.
__global__ void __launch_bounds__(1024) vox_blockscan_kernel(ScanArgs a) {
    __shared__ int sm[32][3];
    const int sc = blockIdx.x;
    const ScaleDev& g = a.s[sc];
    const int nblk = (int)((a.nchunks_used[sc] + kThreads - 1) / kThreads);
    const int per = (nblk + (int)blockDim.x - 1) / (int)blockDim.x;
    const int lo = min(nblk, (int)threadIdx.x * per), hi = min(nblk, lo + per);
    int v[3] = {0, 0, 0}, tot[3];
    for (int i = lo; i < hi; ++i) {
        v[0] += g.blk_sums[i * 3]; v[1] += g.blk_sums[i * 3 + 1]; v[2] += g.blk_sums[i * 3 + 2];
    }
    block_excl_scan3(v, tot, sm);
    for (int i = lo; i < hi; ++i) {
        g.blk_offs[i * 3] = v[0]; g.blk_offs[i * 3 + 1] = v[1]; g.blk_offs[i * 3 + 2] = v[2];
        v[0] += g.blk_sums[i * 3]; v[1] += g.blk_sums[i * 3 + 1]; v[2] += g.blk_sums[i * 3 + 2];
    }
    if (threadIdx.x == 0) {
        g.totals[0] = tot[0]; g.totals[1] = tot[1]; g.totals[2] = tot[2];
        a.num_voxels[sc] = tot[0];
        if (tot[0] > a.capacity[sc]) atomicOr(a.status, kStatusCapacity);
    }
}

// One thread per chunk: rank of the chunk's first voxel, the cell id of every voxel (so that
// later passes can run one thread per voxel), and the bookkeeping of cells over the cap.
__global__ void __launch_bounds__(kThreads) vox_emit_kernel(ScanArgs a) {
    __shared__ int sm[kThreads / 32][3];
    const int sc = blockIdx.y;
    const ScaleDev& g = a.s[sc];
    const uint32_t nblk = (a.nchunks_used[sc] + kThreads - 1) / kThreads;
    if (blockIdx.x >= nblk) return;
    const uint32_t chunk = blockIdx.x * kThreads + threadIdx.x;
    const bool flagged = chunk_flagged(g, chunk, a.nchunks_used[sc]);
    Chunk c;
    int run[3] = {0, 0, 0}, tot[3];
    if (flagged) {
        c = load_chunk(g.store, chunk);
        chunk_stats(g, c, run);
    }
    block_excl_scan3(run, tot, sm);       // run[] = exclusive offsets inside the CTA
    if (!flagged) return;
    int m = g.blk_offs[blockIdx.x * 3] + run[0];
    g.chunk_prefix[chunk] = (uint32_t)m;
    if (g.mode == MODE_BITMAP) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            uint32_t word = c.w[i];
            while (word) {
                const int bit = __ffs(word) - 1;
                word &= word - 1;
                g.cell_list[m++] = chunk * 256u + i * 32u + bit;
            }
        }
    } else {
        int j = g.blk_offs[blockIdx.x * 3 + 1] + run[1];
        int off = g.blk_offs[blockIdx.x * 3 + 2] + run[2];
        if (g.cap > 0) g.chunk_ovf[chunk] = (uint32_t)j;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int n = (int)c.w[i];
            if (n == 0) continue;
            if (g.cap > 0 && n > g.cap) {
                g.ovf_vox[j] = m;
                g.ovf_off[j] = off;
                g.ovf_cursor[j] = 0;
                j += 1;
                off += n;
            }
            g.cell_list[m++] = chunk * 8u + i;
        }
    }
}

// ------------------------------------------------------------------ pass 3: accumulate
struct AccumArgs {
    ScaleDev s[2];
    int capacity[2];
    int32_t* coords[2];
    int32_t* counts[2];
    int32_t* point_voxel[2];
    float* mean[2];
    float* bev;
};

// The first point to arrive in a voxel stores its values in the output row; the others add
// into the fp64 scratch row.  For a count table "first" is decided without an arrival
// counter when the cell holds one point; otherwise an atomic counter elects it.  The kernel
// runs in three phases so that a thread's memory operations overlap: (A) all rank lookups,
// (B) all arrival / list-cursor atomics, (C) all stores and fp64 reductions.
template <int C>
__global__ void __launch_bounds__(kThreads)
vox_accum_kernel(const float* __restrict__ pts, long long total, int N, AccumArgs a) {
    __shared__ __align__(16) float sp[kBigTile * C];
    const long long g0 = (long long)blockIdx.x * kBigTile;
    const int npts = (int)min((long long)kBigTile, total - g0);
    load_tile_f32(pts + g0 * C, npts * C, sp);
    __syncthreads();
    Slot slot[2][kPtsPerThread];
#pragma unroll
    for (int i = 0; i < kPtsPerThread; ++i) {
        const int t = threadIdx.x + i * kThreads;
        uint32_t c0 = 0xFFFFFFFFu, c1 = 0xFFFFFFFFu;
        if (t < npts) {
            const float x = sp[t * C], y = sp[t * C + 1], z = sp[t * C + 2];
            const int b = (int)((g0 + t) / N);
            c0 = cell_of(a.s[0], x, y, z, b);
            c1 = cell_of(a.s[1], x, y, z, b);
        }
        slot[0][i] = slot_of(a.s[0], c0);
        slot[1][i] = slot_of(a.s[1], c1);
    }
    // Phase B.  ticket >= 0: position in arrival order (0 = first); -1: nothing to do.
    // For a cell over the cap the ticket is the slot in its overflow list.
    int ticket[2][kPtsPerThread];
#pragma unroll
    for (int sc = 0; sc < 2; ++sc) {
        const ScaleDev& g = a.s[sc];
#pragma unroll
        for (int i = 0; i < kPtsPerThread; ++i) {
            const Slot s = slot[sc][i];
            int tk = -1;
            if (s.m >= 0) {
                if (s.j >= 0) tk = atomicAdd(&g.ovf_cursor[s.j], 1);
                else if (s.m < a.capacity[sc])
                    tk = (g.mode == MODE_BITMAP || s.n > 1) ? atomicAdd(&g.arrivals[s.m], 1) : 0;
            }
            ticket[sc][i] = tk;
        }
    }
    // Phase C.
#pragma unroll
    for (int sc = 0; sc < 2; ++sc) {
        const ScaleDev& g = a.s[sc];
        float* mean = a.mean[sc];
        int32_t* pv = a.point_voxel[sc];
#pragma unroll
        for (int i = 0; i < kPtsPerThread; ++i) {
            const int t = threadIdx.x + i * kThreads;
            if (t >= npts) continue;
            const Slot s = slot[sc][i];
            const int tk = ticket[sc][i];
            if (s.j >= 0) {
                // Which of this voxel's points survive the cap is decided by vox_overflow_kernel,
                // which also writes their point_voxel entries.
                g.ovf_list[g.ovf_off[s.j] + tk] = (int)(g0 + t);
                continue;
            }
            if (tk == 0) {
#pragma unroll
                for (int k = 0; k < C; ++k) mean[(size_t)s.m * C + k] = sp[t * C + k];
            } else if (tk > 0) {
#pragma unroll
                for (int k = 0; k < C; ++k) atomicAdd(&g.sums[(size_t)s.m * C + k], (double)sp[t * C + k]);
            }
            if (pv) pv[g0 + t] = s.m;
        }
    }
}

// One warp per overflowing voxel: keep the `cap` lowest point indices (keep-first-by-index),
// sum them, and write point_voxel for all of the voxel's points.
template <int C>
__global__ void __launch_bounds__(kThreads)
vox_overflow_kernel(const float* __restrict__ pts, long long total, AccumArgs a, int sc) {
    const ScaleDev& g = a.s[sc];
    const int lane = threadIdx.x & 31;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int nwarps = (gridDim.x * blockDim.x) >> 5;
    const int novf = g.totals[1];
    int32_t* pv = a.point_voxel[sc];
    for (int j = warp; j < novf; j += nwarps) {
        const int m = g.ovf_vox[j];
        const int n = g.ovf_cursor[j];
        const int* list = g.ovf_list + g.ovf_off[j];
        // Smallest t with #{v <= t} >= cap, by bisection on the index value.
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
        if (lane == 0 && m < a.capacity[sc]) {
            // Full sum in scratch; vox_finalize_kernel sees an overflowing cell and ignores
            // the (unwritten) output row.
#pragma unroll
            for (int k = 0; k < C; ++k) g.sums[(size_t)m * C + k] = acc[k];
        }
    }
}

// ------------------------------------------------------------------ pass 4: rows, BEV, cleanup
// One thread per voxel of either scale: coordinates from the cell id, count, mean (first
// arrival + fp64 sums), BEV cell; then the voxel's scratch words go back to zero.  Loads are
// grouped ahead of all stores so that they overlap.
template <int C>
__global__ void __launch_bounds__(kThreads) vox_finalize_kernel(AccumArgs a) {
    const int sc = blockIdx.y;
    const ScaleDev& g = a.s[sc];
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= g.totals[0]) return;
    const bool bitmap = g.mode == MODE_BITMAP;
    const bool in_cap = m < a.capacity[sc];
    float* row = a.mean[sc] + (size_t)m * C;
    double* srow = g.sums + (size_t)m * C;
    // Level 1: everything addressed by m.
    const uint32_t cell = g.cell_list[m];
    const int arr = g.arrivals[m];
    float first[C];
#pragma unroll
    for (int k = 0; k < C; ++k) first[k] = in_cap ? row[k] : 0.0f;
    // Level 2: the cell's point count.
    int n = bitmap ? arr : (int)g.store[cell];
    const bool over = !bitmap && g.cap > 0 && n > g.cap;
    if (over) n = g.cap;
    // Level 3: fp64 sums, only where more than one point contributed.
    const bool use_sums = in_cap && (n > 1 || over);
    double s[C];
#pragma unroll
    for (int k = 0; k < C; ++k) s[k] = use_sums ? srow[k] : 0.0;

    uint32_t r = cell;
    const uint32_t x = r % g.dims[0]; r /= g.dims[0];
    const uint32_t y = r % g.dims[1]; r /= g.dims[1];
    const uint32_t z = r % g.dims[2]; r /= g.dims[2];
    float mu[C];
    const double cnt = (double)n;
#pragma unroll
    for (int k = 0; k < C; ++k)
        mu[k] = use_sums ? (float)((over ? s[k] : s[k] + (double)first[k]) / cnt) : first[k];

    // Stores: cleanup first (also for rows past the caller's capacity), then the outputs.
    if (bitmap) {
        g.store[cell >> 5] = 0u;                       // neighbours in the word write 0 as well
        g.summary[cell >> 13] = 0u;
    } else {
        g.store[cell] = 0u;
        g.summary[cell >> 8] = 0u;
    }
    if (arr) g.arrivals[m] = 0;
    if (!in_cap) return;
    if (use_sums) {
#pragma unroll
        for (int k = 0; k < C; ++k) { srow[k] = 0.0; row[k] = mu[k]; }
    }
    reinterpret_cast<int4*>(a.coords[sc])[m] = make_int4((int)r, (int)z, (int)y, (int)x);
    a.counts[sc][m] = n;
    if (sc == 1 && a.bev) {
        const size_t plane = (size_t)g.dims[1] * g.dims[0];
        float* dst = a.bev + (size_t)r * C * plane + (size_t)y * g.dims[0] + x;
#pragma unroll
        for (int k = 0; k < C; ++k) dst[(size_t)k * plane] = mu[k];
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
    int scan_blocks = 1;
    for (int s = 0; s < 2; ++s) {
        sa.s[s] = h->scale[s];
        aa.s[s] = h->scale[s];
        const uint64_t cells = (uint64_t)B * h->scale[s].cells;
        const uint64_t per_chunk = h->scale[s].mode == MODE_BITMAP ? 256 : 8;
        sa.nchunks_used[s] = (uint32_t)((cells + per_chunk - 1) / per_chunk);
        scan_blocks = max(scan_blocks, (int)((sa.nchunks_used[s] + kThreads - 1) / kThreads));
        sa.capacity[s] = aa.capacity[s] = capacity[s];
        aa.coords[s] = d_coords[s];
        aa.counts[s] = d_counts[s];
        aa.mean[s] = d_mean[s];
        aa.point_voxel[s] = d_point_voxel ? d_point_voxel[s] : nullptr;
    }
    sa.num_voxels = d_num_voxels;
    sa.status = h->d_status;
    aa.bev = d_bev;

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
        LaunchScope ls(h, K_VOX_REDUCE, st);
        vox_reduce_kernel<<<dim3(scan_blocks, 2), kThreads, 0, st>>>(sa);
    }
    {
        LaunchScope ls(h, K_VOX_BLOCKSCAN, st);
        vox_blockscan_kernel<<<2, 1024, 0, st>>>(sa);
    }
    {
        LaunchScope ls(h, K_VOX_EMIT, st);
        vox_emit_kernel<<<dim3(scan_blocks, 2), kThreads, 0, st>>>(sa);
    }
    if (total > 0) {
        {
            LaunchScope ls(h, K_VOX_ACCUM, st);
            vox_accum_kernel<C><<<ptiles, kThreads, 0, st>>>(d_points, total, N, aa);
        }
        for (int s = 0; s < 2; ++s) {
            if (h->scale[s].cap > 0) {
                LaunchScope ls(h, K_VOX_OVERFLOW, st);
                vox_overflow_kernel<C><<<148 * 2, kThreads, 0, st>>>(d_points, total, aa, s);
            }
        }
        {
            // The number of voxels is only known on the device; it cannot exceed the points.
            const int blocks = (int)((total + kThreads - 1) / kThreads);
            LaunchScope ls(h, K_VOX_FINALIZE, st);
            vox_finalize_kernel<C><<<dim3(blocks, 2), kThreads, 0, st>>>(aa);
        }
    }
    return check_cuda(h, cudaGetLastError());
}

}  // namespace

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
