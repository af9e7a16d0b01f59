// Rulebook of a 3 x 3 x 3 submanifold sparse convolution over a voxel list: the index structure of
// the 3D sparse convolution that consumes the voxel lists (Sec. 3.5), built with prefix sums in
// place of an index search (Sec. 3.6).  For kernel offset k = (dz+1)*9 + (dy+1)*3 + (dx+1) the rule
// list holds the pairs (in = n, out = m) with coords[n] = coords[m] + (dz, dy, dx) in the same
// frame, in ascending m.
//
// A neighbour is found in O(1): the scale's direct-addressed cell store (all zero between calls)
// is filled from the list, {32 cell bits, row of the word's first voxel} per 32 cells for large
// grids, the row + 1 per cell for small ones.  Because the list is in cell order, a voxel's row is
// the word's first row plus the number of set bits below it.
//   rb_mark   every voxel sets its cell; the first voxel of a word stores its row there
//   rb_count  27 look-ups per voxel -> neighbour bits per voxel, pair counts per (offset, tile)
//   rb_scan   one CTA per offset: exclusive prefix sum of its counts over the tiles, and its total
//   rb_fill   offsets[28] from the totals; every tile ranks its pairs per offset with warp ballots
//             and writes them
//   rb_clear  the touched words of the store go back to zero
#include "bridge_internal.cuh"

namespace emc2 {
namespace {

constexpr int kStatusCapacity = 1;
constexpr int kStatusBadList = 4;
constexpr int kOffsets = 27;
constexpr int kRbScanThreads = 1024;

struct RbArgs {
    ScaleDev g;
    const int4* coords;          // [capacity] rows (b, z, y, x)
    const int32_t* num_voxels;   // device: voxels in the list
    int capacity, max_batch;
    int tiles;                   // ceil(capacity / kTile)
    uint32_t* nbr_bits;          // [capacity] bit k: the neighbour at offset k exists
    int* tile_counts;            // [27][tiles]
    int* tile_base;              // [27][tiles] exclusive prefix sum of tile_counts along the tiles
    int* offset_pairs;           // [27] pairs per offset
    int32_t* offsets;            // [28]
    int32_t* rule_in;
    int32_t* rule_out;
    long long pair_capacity;
    int* status;
};

__device__ __forceinline__ int voxels_in_list(const RbArgs& a) { return min(*a.num_voxels, a.capacity); }

// Cell id of (b, z, y, x) inside the batch, 0xFFFFFFFF outside the grid.
__device__ __forceinline__ uint32_t cell_at(const RbArgs& a, int b, int z, int y, int x) {
    const ScaleDev& g = a.g;
    if ((unsigned)b >= (unsigned)a.max_batch || (unsigned)z >= (unsigned)g.dims[2] ||
        (unsigned)y >= (unsigned)g.dims[1] || (unsigned)x >= (unsigned)g.dims[0])
        return 0xFFFFFFFFu;
    return (((uint32_t)b * g.dims[2] + z) * g.dims[1] + y) * g.dims[0] + x;
}

__global__ void __launch_bounds__(kThreads) rb_mark_kernel(const __grid_constant__ RbArgs a) {
    const int M = voxels_in_list(a);
    const int m = blockIdx.x * kThreads + threadIdx.x;
    if (m >= M) return;
    const int4 c = a.coords[m];
    const uint32_t cell = cell_at(a, c.x, c.y, c.z, c.w);
    uint32_t before = 0xFFFFFFFFu;
    if (m > 0) {
        const int4 p = a.coords[m - 1];
        before = cell_at(a, p.x, p.y, p.z, p.w);
    }
    // Rows outside the grid, repeated or not in ascending cell order: not a list of this grid.
    if (cell == 0xFFFFFFFFu || (m > 0 && (before == 0xFFFFFFFFu || before >= cell))) {
        atomicOr(a.status, kStatusBadList);
        if (cell == 0xFFFFFFFFu) return;
    }
    if (a.g.mode == MODE_BITMAP) {
        uint32_t* word = a.g.store + 2 * (size_t)(cell >> 5);
        atomicOr(word, 1u << (cell & 31u));
        if (m == 0 || before == 0xFFFFFFFFu || (before >> 5) != (cell >> 5)) word[1] = (uint32_t)m;
    } else {
        a.g.store[4 * (size_t)cell] = (uint32_t)m + 1u;
    }
}

__global__ void __launch_bounds__(kThreads) rb_clear_kernel(const __grid_constant__ RbArgs a) {
    const int M = voxels_in_list(a);
    const int m = blockIdx.x * kThreads + threadIdx.x;
    if (m >= M) return;
    const int4 c = a.coords[m];
    const uint32_t cell = cell_at(a, c.x, c.y, c.z, c.w);
    if (cell == 0xFFFFFFFFu) return;
    if (a.g.mode == MODE_BITMAP) *reinterpret_cast<uint2*>(a.g.store + 2 * (size_t)(cell >> 5)) = make_uint2(0u, 0u);
    else a.g.store[4 * (size_t)cell] = 0u;
}

// Row of the voxel at bit `pos` of a {bits, first row} pair, -1 if the bit is clear.
__device__ __forceinline__ int row_in_word(const uint2 pr, uint32_t pos) {
    const uint32_t bit = 1u << pos;
    return (pr.x & bit) ? (int)(pr.y + __popc(pr.x & (bit - 1u))) : -1;
}

// Where a voxel sits: its cell, the cell strides and which of its 3 x 3 x 3 neighbours the grid has.
struct Site {
    uint32_t cell, sy, sz;
    bool okz[3], oky[3], okx[3];
};

__device__ __forceinline__ Site site_of(const RbArgs& a, const int4 c) {
    const ScaleDev& g = a.g;
    Site s;
    s.cell = cell_at(a, c.x, c.y, c.z, c.w);
    s.sy = (uint32_t)g.dims[0];
    s.sz = s.sy * (uint32_t)g.dims[1];
    s.okz[0] = c.y > 0; s.okz[1] = true; s.okz[2] = c.y + 1 < g.dims[2];
    s.oky[0] = c.z > 0; s.oky[1] = true; s.oky[2] = c.z + 1 < g.dims[1];
    s.okx[0] = c.w > 0; s.okx[1] = true; s.okx[2] = c.w + 1 < g.dims[0];
    return s;
}

// Rows of the three x-neighbours (dx = -1, 0, 1) at (dz, dy) = (j / 3 - 1, j % 3 - 1) of a valid
// site, -1 where there is none; only the ones in `want3` (bit dx + 1) are looked up.  The three
// share a bitmap word unless they straddle a word boundary: one load, rarely two.
__device__ __forceinline__ void neighbours3(const ScaleDev& g, const Site& s, int j, uint32_t want3, int r[3]) {
    const int dz = j / 3 - 1, dy = j % 3 - 1;
    r[0] = r[1] = r[2] = -1;
    if (!want3 || !s.okz[dz + 1] || !s.oky[dy + 1]) return;
    const uint32_t mid = s.cell + (uint32_t)dz * s.sz + (uint32_t)dy * s.sy;   // wraps like the signed sum
    if (g.mode == MODE_BITMAP) {
        const uint2* words = reinterpret_cast<const uint2*>(g.store);
        const uint32_t w = mid >> 5, pos = mid & 31u;
        const uint2 pr = words[w];
        if (want3 & 2u) r[1] = row_in_word(pr, pos);
        if (s.okx[0] && (want3 & 1u)) r[0] = pos > 0 ? row_in_word(pr, pos - 1) : row_in_word(words[w - 1], 31);
        if (s.okx[2] && (want3 & 4u)) r[2] = pos < 31 ? row_in_word(pr, pos + 1) : row_in_word(words[w + 1], 0);
    } else {
#pragma unroll
        for (int i = 0; i < 3; ++i)
            if (s.okx[i] && ((want3 >> i) & 1u)) r[i] = (int)g.store[4 * (size_t)(mid + i - 1)] - 1;
    }
}

// Which of the three x-neighbours at (dz, dy) exist (bit dx + 1), for a valid site.
__device__ __forceinline__ uint32_t exist3(const ScaleDev& g, const Site& s, int j) {
    const int dz = j / 3 - 1, dy = j % 3 - 1;
    if (!s.okz[dz + 1] || !s.oky[dy + 1]) return 0u;
    const uint32_t mid = s.cell + (uint32_t)dz * s.sz + (uint32_t)dy * s.sy;
    const uint32_t inside = (s.okx[0] ? 1u : 0u) | 2u | (s.okx[2] ? 4u : 0u);
    if (g.mode == MODE_BITMAP) {
        const uint32_t w = mid >> 5, pos = mid & 31u;
        // 34-bit window: the word's 32 cells with one cell of the words before and after it
        unsigned long long window = (unsigned long long)g.store[2 * (size_t)w] << 1;
        if (pos == 0 && s.okx[0]) window |= g.store[2 * (size_t)(w - 1)] >> 31;
        if (pos == 31 && s.okx[2]) window |= (unsigned long long)(g.store[2 * (size_t)(w + 1)] & 1u) << 33;
        return (uint32_t)(window >> pos) & inside;
    }
    uint32_t three = 0;
#pragma unroll
    for (int i = 0; i < 3; ++i)
        if (s.okx[i] && g.store[4 * (size_t)(mid + i - 1)]) three |= 1u << i;
    return three;
}

__global__ void __launch_bounds__(kThreads) rb_count_kernel(const __grid_constant__ RbArgs a) {
    __shared__ int wcount[kThreads / 32][kOffsets];
    const int M = voxels_in_list(a);
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int m = blockIdx.x * kTile + t;
    uint32_t bits = 0;
    if (m < M) {
        const int4 c = a.coords[m];
        const Site s = site_of(a, c);
        if (s.cell != 0xFFFFFFFFu) {
#pragma unroll
            for (int j = 0; j < 9; ++j) bits |= exist3(a.g, s, j) << (3 * j);
        }
    }
    if (m < a.capacity) a.nbr_bits[m] = bits;
#pragma unroll
    for (int k = 0; k < kOffsets; ++k) {
        const unsigned b = __ballot_sync(0xFFFFFFFFu, (bits >> k) & 1u);
        if (lane == 0) wcount[warp][k] = __popc(b);
    }
    __syncthreads();
    if (t < kOffsets) {
        int sum = 0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) sum += wcount[w][t];
        a.tile_counts[(size_t)t * a.tiles + blockIdx.x] = sum;
    }
}

// CTA k: exclusive prefix sum of offset k's counts over the tiles, 4096 entries per round, and the
// offset's pair total.  The totals become offsets[28] in rb_fill.
__global__ void __launch_bounds__(kRbScanThreads) rb_scan_kernel(const __grid_constant__ RbArgs a) {
    __shared__ int wsum[kRbScanThreads / 32];
    __shared__ int s_carry;
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int* counts = a.tile_counts + (size_t)blockIdx.x * a.tiles;
    int* base = a.tile_base + (size_t)blockIdx.x * a.tiles;
    if (t == 0) s_carry = 0;
    __syncthreads();
    for (int i0 = 0; i0 < a.tiles; i0 += 4 * kRbScanThreads) {
        const int i = i0 + 4 * t;
        int v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = i + j < a.tiles ? counts[i + j] : 0;
        const int sum = v[0] + v[1] + v[2] + v[3];
        int inc = sum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
            if (lane >= d) inc += y;
        }
        if (lane == 31) wsum[warp] = inc;
        __syncthreads();
        int before = s_carry, round = 0;
        for (int w = 0; w < kRbScanThreads / 32; ++w) {
            if (w < warp) before += wsum[w];
            round += wsum[w];
        }
        int run = before + inc - sum;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (i + j < a.tiles) base[i + j] = run;
            run += v[j];
        }
        __syncthreads();
        if (t == 0) s_carry += round;
        __syncthreads();
    }
    if (t == 0) a.offset_pairs[blockIdx.x] = s_carry;
}

__global__ void __launch_bounds__(kThreads, 6) rb_fill_kernel(const __grid_constant__ RbArgs a) {
    __shared__ int wcount[kThreads / 32][kOffsets];   // pairs per warp, then where the warp's pairs start
    __shared__ int s_start[kOffsets + 1];             // offsets[]
    const int M = voxels_in_list(a);
    if (blockIdx.x > 0 && blockIdx.x * kTile >= M) return;   // CTA 0 always writes offsets[]
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int m = blockIdx.x * kTile + t;
    // Loads that depend on nothing go first.
    const int tile_start = t < kOffsets ? a.tile_base[(size_t)t * a.tiles + blockIdx.x] : 0;
    const int own = t < kOffsets ? a.offset_pairs[t] : 0;
    int4 c = make_int4(0, 0, 0, 0);
    uint32_t bits = 0u;
    if (m < M) {
        c = a.coords[m];
        bits = a.nbr_bits[m];
    }
    if (warp == 0) {                                   // offsets[] from the 27 totals
        int inc = own;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
            if (lane >= d) inc += y;
        }
        if (lane <= kOffsets) s_start[lane] = inc - own;
    }
#pragma unroll
    for (int k = 0; k < kOffsets; ++k) {
        const unsigned b = __ballot_sync(0xFFFFFFFFu, (bits >> k) & 1u);
        if (lane == 0) wcount[warp][k] = __popc(b);
    }
    __syncthreads();
    if (t < kOffsets) {
        int run = s_start[t] + tile_start;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) {
            const int n = wcount[w][t];
            wcount[w][t] = run;
            run += n;
        }
    }
    if (blockIdx.x == 0 && t <= kOffsets) {
        a.offsets[t] = s_start[t];
        if (t == kOffsets && (long long)s_start[t] > a.pair_capacity) atomicOr(a.status, kStatusCapacity);
    }
    __syncthreads();
    const Site s = site_of(a, c);                      // bits == 0 for rows outside the list or the grid
    const unsigned below = (1u << lane) - 1u;
#pragma unroll
    for (int j = 0; j < 9; ++j) {
        int r[3];
        neighbours3(a.g, s, j, (bits >> (3 * j)) & 7u, r);
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const int k = 3 * j + i;
            const bool has = (bits >> k) & 1u;
            const unsigned b = __ballot_sync(0xFFFFFFFFu, has);
            const int pos = wcount[warp][k] + __popc(b & below);
            if (has && (long long)pos < a.pair_capacity) {
                a.rule_in[pos] = r[i];
                a.rule_out[pos] = m;
            }
        }
    }
}

}  // namespace

int launch_rulebook(emc2_bridge* h, int scale, int capacity, const int32_t* d_coords, const int32_t* d_num_voxels,
                    int32_t* d_rule_offsets, int32_t* d_rule_in, int32_t* d_rule_out, long long pair_capacity,
                    cudaStream_t st) {
    RbArgs a;
    a.g = h->scale[scale];
    a.coords = reinterpret_cast<const int4*>(d_coords);
    a.num_voxels = d_num_voxels;
    a.capacity = capacity;
    a.max_batch = h->cfg.max_batch;
    a.tiles = (capacity + kTile - 1) / kTile;
    a.nbr_bits = h->d_rb_bits;
    a.tile_counts = h->d_rb_counts;
    a.tile_base = h->d_rb_base;
    a.offset_pairs = h->d_rb_base + (size_t)kOffsets * a.tiles;
    a.offsets = d_rule_offsets; a.rule_in = d_rule_in; a.rule_out = d_rule_out;
    a.pair_capacity = pair_capacity;
    a.status = h->d_status;
    const unsigned blocks = (unsigned)a.tiles;
    {
        LaunchScope ls(h, K_RB_MARK, st);
        rb_mark_kernel<<<blocks, kThreads, 0, st>>>(a);
    }
    {
        LaunchScope ls(h, K_RB_COUNT, st);
        rb_count_kernel<<<blocks, kThreads, 0, st>>>(a);
    }
    {
        LaunchScope ls(h, K_RB_SCAN, st);
        rb_scan_kernel<<<kOffsets, kRbScanThreads, 0, st>>>(a);
    }
    {
        LaunchScope ls(h, K_RB_FILL, st);
        rb_fill_kernel<<<blocks, kThreads, 0, st>>>(a);
    }
    {
        LaunchScope ls(h, K_RB_CLEAR, st);
        rb_clear_kernel<<<blocks, kThreads, 0, st>>>(a);
    }
    return check_cuda(h, cudaGetLastError());
}

}  // namespace emc2
