// Stage 1 of the bridge: two-scale voxelization, dedup in canonical order, per-voxel counts
// and means, BEV scatter (Sec. 3.1 preprocessing; BEV for the 2D expert of Sec. 3.3).
//
// Dedup is direct-addressed, with no sort: every cell of the batch owns one bit (large grids)
// or one 32-bit counter (grids small enough for a count table).  The store is cut into
// 32-byte chunks (one L2 sector: 256 bitmap cells or 8 counters); a summary bitmap holds one
// bit per chunk.  Points mark their cell with one atomic; a prefix sum over the occupied
// chunks (the parallel prefix-sum index search of Sec. 3.6) then gives every occupied cell its
// rank in ascending (b, z, y, x) order, which is the canonical voxel order.  A second pass
// over the points looks the rank up (one sector load plus popcounts) and accumulates fp64
// sums.  The store is cleaned through the summary bits at the end of the call, so the cost
// follows the occupied cells, not the grid volume.
#include "bridge_internal.cuh"

namespace emc2 {
namespace {

constexpr int kStatusCapacity = 1;
constexpr int kEmitWindow = 2048;   // voxels a CTA stages in shared memory per emission round

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

// Rank of an occupied cell among all occupied cells of the batch (ascending cell id).  For a
// count table also returns the cell's point count and its rank among overflowing cells.
__device__ __forceinline__ uint32_t rank_of(const ScaleDev& g, uint32_t cell, int* n_in_cell, int* ovf_rank) {
    if (g.mode == MODE_BITMAP) {
        const uint32_t chunk = cell >> 8, w = (cell >> 5) & 7u, bit = cell & 31u;
        Chunk c = load_chunk(g.store, chunk);
        uint32_t r = g.chunk_prefix[chunk];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            uint32_t m = i < (int)w ? 0xFFFFFFFFu : (i == (int)w ? ((1u << bit) - 1u) : 0u);
            r += __popc(c.w[i] & m);
        }
        *n_in_cell = 0;
        *ovf_rank = -1;
        return r;
    } else {
        const uint32_t chunk = cell >> 3, w = cell & 7u;
        Chunk c = load_chunk(g.store, chunk);
        uint32_t r = g.chunk_prefix[chunk];
        int before_ovf = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            r += (i < (int)w && c.w[i] != 0u) ? 1u : 0u;
            before_ovf += (i < (int)w && g.cap > 0 && (int)c.w[i] > g.cap) ? 1 : 0;
        }
        const int n = (int)c.w[w];
        *n_in_cell = n;
        *ovf_rank = (g.cap > 0 && n > g.cap) ? (int)g.chunk_ovf[chunk] + before_ovf : -1;
        return r;
    }
}

// ------------------------------------------------------------------ pass 1: mark cells
__device__ __forceinline__ void mark_cell(const ScaleDev& g, float x, float y, float z, int b) {
    const uint32_t cell = cell_of(g, x, y, z, b);
    if (cell == 0xFFFFFFFFu) return;
    uint32_t chunk, old;
    if (g.mode == MODE_BITMAP) {
        old = atomicOr(&g.store[cell >> 5], 1u << (cell & 31u));
        chunk = cell >> 8;
    } else {
        old = atomicAdd(&g.store[cell], 1u);
        chunk = cell >> 3;
    }
    if (old == 0u) atomicOr(&g.summary[chunk >> 5], 1u << (chunk & 31u));
}

template <int C>
__global__ void __launch_bounds__(kThreads)
vox_mark_kernel(const float* __restrict__ pts, long long total, int N, ScaleDev s0, ScaleDev s1) {
    __shared__ __align__(16) float sp[kTile * C];
    const long long g0 = (long long)blockIdx.x * kTile;
    const int npts = (int)min((long long)kTile, total - g0);
    load_tile_f32(pts + g0 * C, npts * C, sp);
    __syncthreads();
    const int t = threadIdx.x;
    if (t >= npts) return;
    const float x = sp[t * C], y = sp[t * C + 1], z = sp[t * C + 2];
    const int b = (int)((g0 + t) / N);
    mark_cell(s0, x, y, z, b);
    mark_cell(s1, x, y, z, b);
}

// ------------------------------------------------------------------ pass 2: ranks
struct ScanArgs {
    ScaleDev s[2];
    uint32_t nchunks_used[2];   // chunks covering this call's B frames
    int capacity[2];
    int32_t* coords[2];
    int32_t* counts[2];
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

// One CTA per scale: exclusive scan of the per-CTA sums; totals, capacity check.
__global__ void __launch_bounds__(1024) vox_blockscan_kernel(ScanArgs a) {
    __shared__ int sm[32][3];
    __shared__ int carry[3];
    const int sc = blockIdx.x;
    const ScaleDev& g = a.s[sc];
    const int nblk = (int)((a.nchunks_used[sc] + kThreads - 1) / kThreads);
    if (threadIdx.x < 3) carry[threadIdx.x] = 0;
    __syncthreads();
    for (int base = 0; base < nblk; base += blockDim.x) {
        const int i = base + threadIdx.x;
        int v[3] = {0, 0, 0}, tot[3];
        if (i < nblk) {
            v[0] = g.blk_sums[i * 3]; v[1] = g.blk_sums[i * 3 + 1]; v[2] = g.blk_sums[i * 3 + 2];
        }
        block_excl_scan3(v, tot, sm);
        if (i < nblk) {
            g.blk_offs[i * 3] = v[0] + carry[0];
            g.blk_offs[i * 3 + 1] = v[1] + carry[1];
            g.blk_offs[i * 3 + 2] = v[2] + carry[2];
        }
        __syncthreads();
        if (threadIdx.x < 3) carry[threadIdx.x] += tot[threadIdx.x];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        g.totals[0] = carry[0]; g.totals[1] = carry[1]; g.totals[2] = carry[2];
        a.num_voxels[sc] = carry[0];
        if (carry[0] > a.capacity[sc]) atomicOr(a.status, kStatusCapacity);
    }
}

// One thread per chunk finds the rank of its first voxel; the CTA then stages its voxels'
// cell ids in shared memory, window by window, and writes the rows of the unique list
// (coords, count, zeroed sums) with consecutive threads on consecutive rows.
template <int C>
__global__ void __launch_bounds__(kThreads) vox_emit_kernel(ScanArgs a) {
    __shared__ int sm[kThreads / 32][3];
    __shared__ uint32_t wcell[kEmitWindow];
    __shared__ int wn[kEmitWindow];
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
    const int m0 = g.blk_offs[blockIdx.x * 3];
    const bool table = g.mode == MODE_TABLE;
    if (flagged) {
        g.chunk_prefix[chunk] = (uint32_t)(m0 + run[0]);
        if (table && g.cap > 0) {
            int j = g.blk_offs[blockIdx.x * 3 + 1] + run[1];
            int off = g.blk_offs[blockIdx.x * 3 + 2] + run[2];
            g.chunk_ovf[chunk] = (uint32_t)j;
            int m = m0 + run[0];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int n = (int)c.w[i];
                if (n > g.cap) {
                    g.ovf_vox[j] = m;
                    g.ovf_off[j] = off;
                    g.ovf_cursor[j] = 0;
                    j += 1;
                    off += n;
                }
                m += n > 0;
            }
        }
    }
    const int cap_rows = a.capacity[sc];
    const uint32_t gx = g.dims[0], gy = g.dims[1], gz = g.dims[2];
    for (int wb = 0; wb < tot[0]; wb += kEmitWindow) {
        if (flagged) {
            int local = run[0] - wb;          // window slot of this chunk's next voxel
            if (table) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (c.w[i]) {
                        if (local >= 0 && local < kEmitWindow) { wcell[local] = chunk * 8u + i; wn[local] = (int)c.w[i]; }
                        local += 1;
                    }
                }
            } else if (local < kEmitWindow) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    uint32_t word = c.w[i];
                    while (word) {
                        const int bit = __ffs(word) - 1;
                        word &= word - 1;
                        if (local >= 0 && local < kEmitWindow) wcell[local] = chunk * 256u + i * 32u + bit;
                        local += 1;
                    }
                }
            }
        }
        __syncthreads();
        const int nw = min(kEmitWindow, tot[0] - wb);
        for (int i = threadIdx.x; i < nw; i += kThreads) {
            const int m = m0 + wb + i;
            if (m < cap_rows) {
                uint32_t cell = wcell[i];
                const uint32_t x = cell % gx; cell /= gx;
                const uint32_t y = cell % gy; cell /= gy;
                const uint32_t z = cell % gz; cell /= gz;
                reinterpret_cast<int4*>(a.coords[sc])[m] = make_int4((int)cell, (int)z, (int)y, (int)x);
                int cnt = 0;
                if (table) cnt = (g.cap > 0 && wn[i] > g.cap) ? g.cap : wn[i];
                a.counts[sc][m] = cnt;
#pragma unroll
                for (int k = 0; k < C; ++k) g.sums[(size_t)m * C + k] = 0.0;
            }
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------ pass 3: accumulate
template <int C>
__device__ __forceinline__ void accum_point(const ScaleDev& g, const float* p, int b, long long gi,
                                            int cap_rows, int32_t* counts, int32_t* point_voxel) {
    const uint32_t cell = cell_of(g, p[0], p[1], p[2], b);
    int pv = -1;
    if (cell != 0xFFFFFFFFu) {
        int n, j;
        const int m = (int)rank_of(g, cell, &n, &j);
        if (j >= 0) {
            // Which of this voxel's points survive the cap is decided by vox_overflow_kernel.
            const int slot = g.ovf_off[j] + atomicAdd(&g.ovf_cursor[j], 1);
            g.ovf_list[slot] = (int)gi;
            return;
        }
        pv = m;
        if (m < cap_rows) {
            if (g.mode == MODE_BITMAP) atomicAdd(&counts[m], 1);
#pragma unroll
            for (int k = 0; k < C; ++k) atomicAdd(&g.sums[(size_t)m * C + k], (double)p[k]);
        }
    }
    if (point_voxel) point_voxel[gi] = pv;
}

struct AccumArgs {
    ScaleDev s[2];
    int capacity[2];
    int32_t* counts[2];
    int32_t* point_voxel[2];
    float* mean[2];
    const int32_t* coords[2];
    float* bev;
    int B;
};

template <int C>
__global__ void __launch_bounds__(kThreads)
vox_accum_kernel(const float* __restrict__ pts, long long total, int N, AccumArgs a) {
    __shared__ __align__(16) float sp[kTile * C];
    const long long g0 = (long long)blockIdx.x * kTile;
    const int npts = (int)min((long long)kTile, total - g0);
    load_tile_f32(pts + g0 * C, npts * C, sp);
    __syncthreads();
    const int t = threadIdx.x;
    if (t >= npts) return;
    float p[C];
#pragma unroll
    for (int k = 0; k < C; ++k) p[k] = sp[t * C + k];
    const long long gi = g0 + t;
    const int b = (int)(gi / N);
    accum_point<C>(a.s[0], p, b, gi, a.capacity[0], a.counts[0], a.point_voxel[0]);
    accum_point<C>(a.s[1], p, b, gi, a.capacity[1], a.counts[1], a.point_voxel[1]);
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
#pragma unroll
            for (int k = 0; k < C; ++k) g.sums[(size_t)m * C + k] = acc[k];
        }
    }
}

// ------------------------------------------------------------------ pass 4: means, BEV
template <int C>
__global__ void __launch_bounds__(kThreads) vox_finalize_kernel(AccumArgs a, int rows0, int rows1) {
    const int sc = blockIdx.y;
    const ScaleDev& g = a.s[sc];
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    const int rows = min(min(sc ? rows1 : rows0, g.totals[0]), a.capacity[sc]);
    if (m >= rows) return;
    const double cnt = (double)a.counts[sc][m];
    float mu[C];
#pragma unroll
    for (int k = 0; k < C; ++k) {
        mu[k] = (float)(g.sums[(size_t)m * C + k] / cnt);
        a.mean[sc][(size_t)m * C + k] = mu[k];
    }
    if (sc == 1 && a.bev) {
        const int4 c = reinterpret_cast<const int4*>(a.coords[1])[m];   // (b, z, y, x)
        const size_t plane = (size_t)g.dims[1] * g.dims[0];
        float* dst = a.bev + (size_t)c.x * C * plane + (size_t)c.z * g.dims[0] + c.w;
#pragma unroll
        for (int k = 0; k < C; ++k) dst[(size_t)k * plane] = mu[k];
    }
}

// ------------------------------------------------------------------ pass 5: clean the store
__global__ void __launch_bounds__(kThreads) vox_clean_kernel(ScanArgs a) {
    const int sc = blockIdx.y;
    const ScaleDev& g = a.s[sc];
    const uint32_t nwords = (a.nchunks_used[sc] + 31) / 32;
    const uint32_t wi = blockIdx.x * kThreads + threadIdx.x;
    if (wi >= nwords) return;
    uint32_t sumword = g.summary[wi];
    if (!sumword) return;
    g.summary[wi] = 0u;
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    while (sumword) {
        const int bit = __ffs(sumword) - 1;
        sumword &= sumword - 1;
        uint4* p = reinterpret_cast<uint4*>(g.store + (size_t)(wi * 32u + bit) * 8);
        p[0] = z;
        p[1] = z;
    }
}

__global__ void __launch_bounds__(kThreads) zero_f4_kernel(float4* p, size_t n4) {
    const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x)
        p[i] = z;
}

template <int C>
int run_voxelize(emc2_bridge* h, int B, int N, const float* d_points, int32_t* const d_coords[2],
                 int32_t* const d_counts[2], float* const d_mean[2], int32_t* const d_point_voxel[2],
                 const int32_t capacity[2], int32_t* d_num_voxels, float* d_bev, cudaStream_t st) {
    const long long total = (long long)B * N;
    const int ptiles = (int)((total + kTile - 1) / kTile);
    ScanArgs sa;
    AccumArgs aa;
    int scan_blocks = 1, clean_blocks = 1;
    for (int s = 0; s < 2; ++s) {
        sa.s[s] = h->scale[s];
        aa.s[s] = h->scale[s];
        const uint64_t cells = (uint64_t)B * h->scale[s].cells;
        const uint64_t per_chunk = h->scale[s].mode == MODE_BITMAP ? 256 : 8;
        sa.nchunks_used[s] = (uint32_t)((cells + per_chunk - 1) / per_chunk);
        scan_blocks = max(scan_blocks, (int)((sa.nchunks_used[s] + kThreads - 1) / kThreads));
        clean_blocks = max(clean_blocks, (int)(((sa.nchunks_used[s] + 31) / 32 + kThreads - 1) / kThreads));
        sa.capacity[s] = aa.capacity[s] = capacity[s];
        sa.coords[s] = d_coords[s];
        sa.counts[s] = aa.counts[s] = d_counts[s];
        aa.coords[s] = d_coords[s];
        aa.mean[s] = d_mean[s];
        aa.point_voxel[s] = d_point_voxel ? d_point_voxel[s] : nullptr;
    }
    sa.num_voxels = d_num_voxels;
    sa.status = h->d_status;
    aa.bev = d_bev;
    aa.B = B;

    if (d_bev && B > 0) {
        const size_t n = (size_t)B * C * h->scale[1].dims[1] * h->scale[1].dims[0];
        LaunchScope ls(h, K_BEV_ZERO, st);
        if ((n & 3) == 0) {
            zero_f4_kernel<<<148 * 8, kThreads, 0, st>>>(reinterpret_cast<float4*>(d_bev), n >> 2);
        } else {
            cudaMemsetAsync(d_bev, 0, n * sizeof(float), st);
        }
    }
    if (total > 0) {
        LaunchScope ls(h, K_VOX_MARK, st);
        vox_mark_kernel<C><<<ptiles, kThreads, 0, st>>>(d_points, total, N, sa.s[0], sa.s[1]);
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
        vox_emit_kernel<C><<<dim3(scan_blocks, 2), kThreads, 0, st>>>(sa);
    }
    if (total > 0) {
        LaunchScope ls(h, K_VOX_ACCUM, st);
        vox_accum_kernel<C><<<ptiles, kThreads, 0, st>>>(d_points, total, N, aa);
    }
    for (int s = 0; s < 2; ++s) {
        if (h->scale[s].cap > 0 && total > 0) {
            LaunchScope ls(h, K_VOX_OVERFLOW, st);
            vox_overflow_kernel<C><<<148 * 2, kThreads, 0, st>>>(d_points, total, aa, s);
        }
    }
    {
        const long long r0 = min((long long)capacity[0], total), r1 = min((long long)capacity[1], total);
        const int blocks = (int)((max(r0, r1) + kThreads - 1) / kThreads);
        if (blocks > 0) {
            LaunchScope ls(h, K_VOX_FINALIZE, st);
            vox_finalize_kernel<C><<<dim3(blocks, 2), kThreads, 0, st>>>(aa, (int)r0, (int)r1);
        }
    }
    {
        LaunchScope ls(h, K_VOX_CLEAN, st);
        vox_clean_kernel<<<dim3(clean_blocks, 2), kThreads, 0, st>>>(sa);
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
