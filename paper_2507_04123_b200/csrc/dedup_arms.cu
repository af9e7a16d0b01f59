// Two alternative designs of the voxel dedup, built to be measured beside the direct-addressed
// cell store of voxelize.cu (same outputs, bit for bit; chosen per scale with
// emc2_bridge_set_tuning):
//
//   sort   every point's cell id and index are sorted by cell id with a stable LSD radix sort
//          (8-bit digits); runs of equal ids are the voxels, in canonical (ascending id) order, and
//          an exclusive prefix sum over the run heads is the voxel row (Sec. 3.6's prefix-sum
//          indexing on sorted keys).
//   hash   the cell ids are deduplicated in an open-addressing table in HBM, sized by the points
//          (linear probing, a bounded number of probes, insertion by compare-and-swap); a hash
//          table has no order, so the unique ids are then sorted with the same radix sort and the
//          position of an id in the sorted list is its row, which goes back into the table for
//          the points to look up.
//
// Both leave what the rest of stage 1 needs: the number of voxels, the list of their cell ids in
// row order, every point's row (or -1), and zeroed accumulators.  The accumulate and finalize
// passes of voxelize.cu then run unchanged.  Neither design spins on another CTA: a probe
// sequence that runs out sets the sticky status word and treats the point as outside the grid.
#include "bridge_internal.cuh"

namespace emc2 {
namespace {

constexpr uint32_t kNoCell = 0xFFFFFFFFu;
constexpr int kSortItems = 8;                       // items per thread of a radix-sort tile
constexpr int kSortTile = kThreads * kSortItems;    // 2,048 items per CTA
constexpr int kScanThreads1 = 1024;
constexpr int kMaxProbes = 128;
constexpr int kStatusCapacity = 1;
constexpr int kStatusProbes = 8;                    // reported as EMC2_ERR_INTERNAL

// ---------------------------------------------------------------- cell ids of the points
template <int C>
__global__ void __launch_bounds__(kThreads)
arm_keys_kernel(const float* __restrict__ pts, long long total, int N, ScaleDev g, uint32_t* keys, uint32_t* vals) {
    const long long i = (long long)blockIdx.x * kThreads + threadIdx.x;
    if (i >= total) return;
    const float* p = pts + i * C;
    keys[i] = cell_of(g, __ldg(p), __ldg(p + 1), __ldg(p + 2), (int)(i / N));
    if (vals) vals[i] = (uint32_t)i;
}

// ---------------------------------------------------------------- stable LSD radix sort, one pass
// counts[d * tiles + tile] = items of the tile whose digit is d.
__global__ void __launch_bounds__(kThreads)
rs_hist_kernel(const uint32_t* __restrict__ keys, int n, int shift, int tiles, int* counts) {
    __shared__ int hist[256];
    const int t = threadIdx.x, tile = blockIdx.x;
    hist[t] = 0;
    __syncthreads();
#pragma unroll
    for (int r = 0; r < kSortItems; ++r) {
        const int i = tile * kSortTile + r * kThreads + t;
        if (i < n) atomicAdd(&hist[(keys[i] >> shift) & 255u], 1);
    }
    __syncthreads();
    counts[t * tiles + tile] = hist[t];
}

// Exclusive prefix sum of `len` ints in place, by one CTA; the grand total goes to *total_out if
// given.  Every thread owns a run of consecutive entries.
__global__ void __launch_bounds__(kScanThreads1) excl_scan_kernel(int* data, int len, int* total_out) {
    constexpr int kWarps = kScanThreads1 / 32;
    __shared__ int wsum[kWarps];
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int per = (len + kScanThreads1 - 1) / kScanThreads1;
    const int lo = min(len, t * per), hi = min(len, lo + per);
    int sum = 0;
    for (int i = lo; i < hi; ++i) sum += data[i];
    int inc = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= d) inc += y;
    }
    if (lane == 31) wsum[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int x = wsum[lane];
        const int v = x;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xFFFFFFFFu, x, d);
            if (lane >= d) x += y;
        }
        wsum[lane] = x - v;
        if (lane == 31 && total_out) *total_out = x;
    }
    __syncthreads();
    int run = wsum[warp] + inc - sum;
    for (int i = lo; i < hi; ++i) {
        const int v = data[i];
        data[i] = run;
        run += v;
    }
}

// CTA d turns row d of counts[256][tiles] (the tiles' counts of digit d) into its exclusive prefix sum
// and leaves the row's total in row_tot[d]; 256-entry chunks with a running carry.
__global__ void __launch_bounds__(kThreads) rs_rowscan_kernel(int* counts, int tiles, int* row_tot) {
    __shared__ int wsum[kThreads / 32];
    __shared__ int s_carry;
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    int* row = counts + (size_t)blockIdx.x * tiles;
    if (t == 0) s_carry = 0;
    __syncthreads();
    for (int c0 = 0; c0 < tiles; c0 += kThreads) {
        const int i = c0 + t;
        const int v = i < tiles ? row[i] : 0;
        int inc = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
            if (lane >= d) inc += y;
        }
        if (lane == 31) wsum[warp] = inc;
        __syncthreads();
        int before = s_carry, all = 0;
        for (int w = 0; w < kThreads / 32; ++w) {
            if (w < warp) before += wsum[w];
            all += wsum[w];
        }
        if (i < tiles) row[i] = before + inc - v;
        __syncthreads();
        if (t == 0) s_carry += all;
        __syncthreads();
    }
    if (t == 0) row_tot[blockIdx.x] = s_carry;
}

// Moves the tile's items to their places.  The tile is taken in rounds of 256 consecutive items, one
// per thread, so that "earlier in the array" is "earlier round, or lower thread": inside a round the
// rank among equal digits comes from a warp match (lanes below) plus the counts of the warps before.
__global__ void __launch_bounds__(kThreads)
rs_scatter_kernel(const uint32_t* __restrict__ keys_in, const uint32_t* __restrict__ vals_in, uint32_t* keys_out,
                  uint32_t* vals_out, int n, int shift, int tiles, const int* __restrict__ bases,
                  const int* __restrict__ row_tot) {
    constexpr int kWarps = kThreads / 32;
    __shared__ int base[256];
    __shared__ int wcnt[kWarps][256];
    __shared__ int dsum[kWarps];
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5, tile = blockIdx.x;
    {
        // Items of smaller digits anywhere (exclusive prefix of the digit totals) + items of this digit in
        // earlier tiles.
        const int v = row_tot[t];
        int inc = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
            if (lane >= d) inc += y;
        }
        if (lane == 31) dsum[warp] = inc;
        __syncthreads();
        int before = 0;
        for (int w = 0; w < warp; ++w) before += dsum[w];
        base[t] = before + inc - v + bases[t * tiles + tile];
    }
    for (int r = 0; r < kSortItems; ++r) {
#pragma unroll
        for (int w = 0; w < kWarps; ++w) wcnt[w][t] = 0;
        __syncthreads();
        const int i = tile * kSortTile + r * kThreads + t;
        const bool valid = i < n;
        uint32_t key = 0u, val = 0u;
        int d = -1;
        if (valid) {
            key = keys_in[i];
            if (vals_in) val = vals_in[i];
            d = (int)((key >> shift) & 255u);
        }
        const unsigned peers = __match_any_sync(0xFFFFFFFFu, d);
        const int lrank = __popc(peers & ((1u << lane) - 1u));
        if (valid && lrank == 0) wcnt[warp][d] = __popc(peers);
        __syncthreads();
        if (valid) {
            int pos = base[d] + lrank;
            for (int w = 0; w < warp; ++w) pos += wcnt[w][d];
            keys_out[pos] = key;
            if (vals_out) vals_out[pos] = val;
        }
        __syncthreads();
        int tot = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) tot += wcnt[w][t];
        base[t] += tot;
        __syncthreads();
    }
}

// ---------------------------------------------------------------- sort design: runs of equal ids
// flags of run heads per 1,024-item tile -> tile_tot
constexpr int kHeadTile = 1024;

__device__ __forceinline__ bool is_head(const uint32_t* keys, int i) {
    const uint32_t k = keys[i];
    return k != kNoCell && (i == 0 || keys[i - 1] != k);
}

__global__ void __launch_bounds__(kThreads) head_count_kernel(const uint32_t* __restrict__ keys, int n, int* tile_tot) {
    __shared__ int wsum[kThreads / 32];
    const int t = threadIdx.x;
    int c = 0;
#pragma unroll
    for (int r = 0; r < kHeadTile / kThreads; ++r) {
        const int i = blockIdx.x * kHeadTile + r * kThreads + t;
        if (i < n && is_head(keys, i)) ++c;
    }
    c = warp_sum(c);
    if ((t & 31) == 0) wsum[t >> 5] = c;
    __syncthreads();
    if (t == 0) {
        int v = 0;
        for (int w = 0; w < kThreads / 32; ++w) v += wsum[w];
        tile_tot[blockIdx.x] = v;
    }
}

struct ArmOut {
    uint32_t* cell_list;    // [max_list] cell id of every voxel, ascending
    int* point_rank;        // [total] row of every point's voxel, -1 if outside
    int* totals;            // the scale's totals (as the rank scan of voxelize.cu leaves them)
    int32_t* num_voxels;    // the caller's entry for this scale
    int* status;
    float4* acc;            // accumulators to clear, two float4 per voxel
    int capacity;
    uint32_t max_list;
};

// tile_base = exclusive prefix of tile_tot.  Row of sorted item i = heads before i, minus one for a
// non-head (it belongs to the run that started before it).
__global__ void __launch_bounds__(kThreads)
head_assign_kernel(const uint32_t* __restrict__ keys, const uint32_t* __restrict__ idx, int n,
                   const int* __restrict__ tile_base, ArmOut o) {
    __shared__ int wsum[kThreads / 32];
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    int run = tile_base[blockIdx.x];
    for (int r = 0; r < kHeadTile / kThreads; ++r) {
        const int i = blockIdx.x * kHeadTile + r * kThreads + t;
        const bool in = i < n;
        const uint32_t k = in ? keys[i] : kNoCell;
        const bool head = in && is_head(keys, i);
        const unsigned hm = __ballot_sync(0xFFFFFFFFu, head);
        if (lane == 0) wsum[warp] = __popc(hm);
        __syncthreads();
        int before = 0, all = 0;
        for (int w = 0; w < kThreads / 32; ++w) {
            if (w < warp) before += wsum[w];
            all += wsum[w];
        }
        const int heads_upto = run + before + __popc(hm & ((2u << lane) - 1u));   // heads at or before i
        if (in) {
            const int m = k == kNoCell ? -1 : heads_upto - 1;
            o.point_rank[idx[i]] = m;
            if (head && (uint32_t)m < o.max_list) o.cell_list[m] = k;
        }
        run += all;
        __syncthreads();
    }
}

// Totals, status and cleared accumulators once the number of voxels is known (in *d_total).
__global__ void __launch_bounds__(kThreads) arm_finish_kernel(const int* d_total, ArmOut o) {
    const int M = *d_total;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        o.totals[0] = M; o.totals[1] = 0; o.totals[2] = 0; o.totals[3] = 0;
        *o.num_voxels = M;
        if (M > o.capacity) atomicOr(o.status, kStatusCapacity);
    }
    const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    const size_t n = 2 * (size_t)min((uint32_t)M, o.max_list);
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += (size_t)gridDim.x * kThreads) o.acc[i] = z;
}

// ---------------------------------------------------------------- hash design
__device__ __forceinline__ uint32_t hash_cell(uint32_t k) {      // a 32-bit finaliser (multiply-xorshift)
    k ^= k >> 16; k *= 0x7FEB352Du; k ^= k >> 15; k *= 0x846CA68Bu; k ^= k >> 16;
    return k;
}

// Inserts every point's cell id.  The point that inserted an id (its compare-and-swap found the slot
// empty) also writes the id at its own place of `first`, every other point writes "none": `first`
// then holds each unique id exactly once, ready to be sorted.
__global__ void __launch_bounds__(kThreads)
hash_insert_kernel(const uint32_t* __restrict__ keys, int n, uint32_t* tab_keys, uint32_t mask, uint32_t* first,
                   int* status) {
    const int i = blockIdx.x * kThreads + threadIdx.x;
    if (i >= n) return;
    const uint32_t k = keys[i];
    uint32_t mine = kNoCell;
    if (k != kNoCell) {
        uint32_t h = hash_cell(k) & mask;
        int probe = 0;
        for (; probe < kMaxProbes; ++probe) {
            const uint32_t seen = tab_keys[h];
            if (seen == k) break;
            if (seen == kNoCell) {
                const uint32_t old = atomicCAS(&tab_keys[h], kNoCell, k);
                if (old == kNoCell) { mine = k; break; }
                if (old == k) break;
            }
            h = (h + 1) & mask;
        }
        if (probe == kMaxProbes) atomicOr(status, kStatusProbes);
    }
    first[i] = mine;
}

// Sorted unique ids -> number of voxels (the ids end where "none" begins), cell list, and the row of
// every id stored beside it in the table.
__global__ void __launch_bounds__(kThreads)
hash_assign_kernel(const uint32_t* __restrict__ sorted, int n, const uint32_t* __restrict__ tab_keys, int* tab_rows,
                   uint32_t mask, int* d_total, ArmOut o) {
    const int j = blockIdx.x * kThreads + threadIdx.x;
    if (j >= n) return;
    const uint32_t k = sorted[j];
    if (k == kNoCell) {
        if (j == 0) *d_total = 0;
        return;
    }
    if (j + 1 == n || sorted[j + 1] == kNoCell) *d_total = j + 1;
    if ((uint32_t)j < o.max_list) o.cell_list[j] = k;
    uint32_t h = hash_cell(k) & mask;
    for (int probe = 0; probe < kMaxProbes; ++probe) {
        if (tab_keys[h] == k) { tab_rows[h] = j; return; }
        h = (h + 1) & mask;
    }
}

__global__ void __launch_bounds__(kThreads)
hash_lookup_kernel(const uint32_t* __restrict__ keys, int n, const uint32_t* __restrict__ tab_keys,
                   const int* __restrict__ tab_rows, uint32_t mask, int* point_rank) {
    const int i = blockIdx.x * kThreads + threadIdx.x;
    if (i >= n) return;
    const uint32_t k = keys[i];
    int m = -1;
    if (k != kNoCell) {
        uint32_t h = hash_cell(k) & mask;
        for (int probe = 0; probe < kMaxProbes; ++probe) {
            const uint32_t seen = tab_keys[h];
            if (seen == k) { m = tab_rows[h]; break; }
            if (seen == kNoCell) break;               // a point whose probe sequence ran out: outside
            h = (h + 1) & mask;
        }
    }
    point_rank[i] = m;
}

int key_bits(uint64_t cells_in_call) {               // bits that tell every cell id AND "none" apart
    int bits = 1;
    while (bits < 32 && ((uint64_t)1 << bits) < cells_in_call + 1) ++bits;
    return bits;
}

// Sorts n (key, value) pairs by the low `bits` bits of the key; returns which buffer holds the result.
int radix_sort(emc2_bridge* h, int n, int bits, uint32_t* keys[2], uint32_t* vals[2], bool with_vals, cudaStream_t st) {
    const int tiles = (n + kSortTile - 1) / kSortTile;
    int cur = 0;
    for (int shift = 0; shift < bits; shift += 8) {
        {
            LaunchScope ls(h, K_ARM_SORT, st);
            rs_hist_kernel<<<tiles, kThreads, 0, st>>>(keys[cur], n, shift, tiles, h->arm.counts);
            rs_rowscan_kernel<<<256, kThreads, 0, st>>>(h->arm.counts, tiles, h->arm.row_tot);
            rs_scatter_kernel<<<tiles, kThreads, 0, st>>>(keys[cur], with_vals ? vals[cur] : nullptr, keys[cur ^ 1],
                                                          with_vals ? vals[cur ^ 1] : nullptr, n, shift, tiles,
                                                          h->arm.counts, h->arm.row_tot);
        }
        cur ^= 1;
    }
    return cur;
}

}  // namespace

int dedup_arm_alloc(emc2_bridge* h) {
    if (h->arm.slab) return EMC2_OK;
    const size_t n = (size_t)h->cfg.max_batch * h->cfg.max_points;
    const size_t tiles = (n + kSortTile - 1) / kSortTile;
    const size_t head_tiles = (n + kHeadTile - 1) / kHeadTile;
    size_t slots = 1;
    while (slots < 2 * n) slots <<= 1;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t o = off; off += (bytes + 255) & ~(size_t)255; return o; };
    const size_t o_k0 = take(n * 4), o_k1 = take(n * 4), o_v0 = take(n * 4), o_v1 = take(n * 4);
    const size_t o_counts = take(256 * tiles * 4), o_tt = take((head_tiles + 1) * 4);
    const size_t o_pr0 = take(n * 4), o_pr1 = take(n * 4);
    const size_t o_tk = take(slots * 4), o_tr = take(slots * 4), o_tot = take(16), o_rt = take(256 * 4);
    void* p = nullptr;
    if (cudaMalloc(&p, off) != cudaSuccess) return EMC2_ERR_CUDA;
    char* base = static_cast<char*>(p);
    h->arm.slab = p;
    h->arm.bytes = off;
    h->arm.keys[0] = reinterpret_cast<uint32_t*>(base + o_k0); h->arm.keys[1] = reinterpret_cast<uint32_t*>(base + o_k1);
    h->arm.vals[0] = reinterpret_cast<uint32_t*>(base + o_v0); h->arm.vals[1] = reinterpret_cast<uint32_t*>(base + o_v1);
    h->arm.counts = reinterpret_cast<int*>(base + o_counts);
    h->arm.tile_tot = reinterpret_cast<int*>(base + o_tt);
    h->arm.point_rank[0] = reinterpret_cast<int*>(base + o_pr0); h->arm.point_rank[1] = reinterpret_cast<int*>(base + o_pr1);
    h->arm.tab_keys = reinterpret_cast<uint32_t*>(base + o_tk);
    h->arm.tab_rows = reinterpret_cast<int*>(base + o_tr);
    h->arm.d_total = reinterpret_cast<int*>(base + o_tot);
    h->arm.row_tot = reinterpret_cast<int*>(base + o_rt);
    h->arm.slots = (uint32_t)slots;
    return EMC2_OK;
}

// Dedup of scale `s` by design 1 (hash) or 2 (sort); see the header of this file for what it leaves.
int launch_dedup_arm(emc2_bridge* h, int s, int design, int B, int N, const float* d_points, int capacity,
                     int32_t* d_num_voxels, cudaStream_t st) {
    if (!h->arm.slab) return EMC2_ERR_INTERNAL;
    const int n = B * N;
    const ScaleDev& g = h->scale[s];
    ArmOut o;
    o.cell_list = g.cell_list; o.point_rank = h->arm.point_rank[s]; o.totals = g.totals;
    o.num_voxels = d_num_voxels + s; o.status = h->d_status; o.acc = g.acc; o.capacity = capacity;
    o.max_list = g.max_list;
    const int fin_blocks = 2 * h->num_sms;
    if (n == 0) {
        LaunchScope ls(h, K_ARM_RANK, st);
        cudaMemsetAsync(h->arm.d_total, 0, sizeof(int), st);
        arm_finish_kernel<<<1, kThreads, 0, st>>>(h->arm.d_total, o);
        return check_cuda(h, cudaGetLastError());
    }
    const int blocks = (n + kThreads - 1) / kThreads;
    const int bits = key_bits((uint64_t)B * g.cells);
    {
        LaunchScope ls(h, K_ARM_KEYS, st);
        if (h->cfg.point_floats == 4)
            arm_keys_kernel<4><<<blocks, kThreads, 0, st>>>(d_points, n, N, g, h->arm.keys[0], design == 2 ? h->arm.vals[0] : nullptr);
        else
            arm_keys_kernel<5><<<blocks, kThreads, 0, st>>>(d_points, n, N, g, h->arm.keys[0], design == 2 ? h->arm.vals[0] : nullptr);
    }
    if (design == 2) {
        const int cur = radix_sort(h, n, bits, h->arm.keys, h->arm.vals, true, st);
        const int head_tiles = (n + kHeadTile - 1) / kHeadTile;
        LaunchScope ls(h, K_ARM_RANK, st);
        head_count_kernel<<<head_tiles, kThreads, 0, st>>>(h->arm.keys[cur], n, h->arm.tile_tot);
        excl_scan_kernel<<<1, kScanThreads1, 0, st>>>(h->arm.tile_tot, head_tiles, h->arm.d_total);
        head_assign_kernel<<<head_tiles, kThreads, 0, st>>>(h->arm.keys[cur], h->arm.vals[cur], n, h->arm.tile_tot, o);
        arm_finish_kernel<<<fin_blocks, kThreads, 0, st>>>(h->arm.d_total, o);
    } else {
        // keys[0] keeps the points' ids for the look-up; the unique ids are sorted in vals[0] / vals[1].
        {
            LaunchScope ls(h, K_ARM_HASH, st);
            cudaMemsetAsync(h->arm.tab_keys, 0xFF, (size_t)h->arm.slots * 4, st);
            hash_insert_kernel<<<blocks, kThreads, 0, st>>>(h->arm.keys[0], n, h->arm.tab_keys, h->arm.slots - 1,
                                                            h->arm.vals[0], h->d_status);
        }
        const int cur = radix_sort(h, n, bits, h->arm.vals, h->arm.keys, false, st);
        LaunchScope ls(h, K_ARM_RANK, st);
        hash_assign_kernel<<<blocks, kThreads, 0, st>>>(h->arm.vals[cur], n, h->arm.tab_keys, h->arm.tab_rows,
                                                        h->arm.slots - 1, h->arm.d_total, o);
        hash_lookup_kernel<<<blocks, kThreads, 0, st>>>(h->arm.keys[0], n, h->arm.tab_keys, h->arm.tab_rows,
                                                        h->arm.slots - 1, o.point_rank);
        arm_finish_kernel<<<fin_blocks, kThreads, 0, st>>>(h->arm.d_total, o);
    }
    return check_cuda(h, cudaGetLastError());
}

}  // namespace emc2
