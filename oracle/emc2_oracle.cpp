// CPU oracle for the EMC2 data bridge and dispatch (test infrastructure only).
//
// A plain, single-threaded, deliberately slow restatement of what the bridge
// computes before any expert model runs (Adaptive Multimodal Data Bridge,
// Sec. 3.1; Scenario-Adaptive Dispatcher, Sec. 3.2; fusion rule of Fig. 5;
// prefix-sum indexing, Sec. 3.6).  It exists so that tests and the benchmark's
// CPU-baseline leg have an independent answer to compare the CUDA library
// with.  It shares no code with that library, is never linked into it, and no
// product path may call it.
//
// Build: g++ -std=c++17 -O2 -ffp-contract=off (no fast-math), so every fp32
// operation below is a single IEEE round-to-nearest operation in the order
// written.  Every function is pinned by tests against closed forms, brute
// force and library special cases; none is "parity unpinned".
//
// Conventions: points are row-major float32 [B, N, C] with (x, y, z) first;
// all indices are 32-bit; a "frame" is one b in [0, B).
#include <algorithm>
#include <array>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <map>
#include <vector>

namespace {

// Voxel index along one axis (Sec. 3.1 names voxelization but gives no
// formula; this is the usual floor((p - min) / size) with one fp32 subtract
// and one fp32 divide).  Returns -1 when the point is outside [0, dim).
int axis_index(float p, float mn, float size, int dim) {
    if (!std::isfinite(p)) return -1;
    float d = p - mn;
    float q = d / size;
    float f = std::floor(q);
    if (!(f >= 0.0f)) return -1;              // also rejects NaN
    if (!(f < (float)dim)) return -1;
    return (int)f;
}

// Linear key of a cell inside the whole batch: ((b*Gz + iz)*Gy + iy)*Gx + ix.
// Ascending key order == ascending (b, z, y, x).
bool voxel_key(const float* p, int b, const float mn[3], const float vs[3], const int dims[3],
               uint64_t* key) {
    int ix = axis_index(p[0], mn[0], vs[0], dims[0]);
    int iy = axis_index(p[1], mn[1], vs[1], dims[1]);
    int iz = axis_index(p[2], mn[2], vs[2], dims[2]);
    if (ix < 0 || iy < 0 || iz < 0) return false;
    *key = (((uint64_t)b * (uint64_t)dims[2] + (uint64_t)iz) * (uint64_t)dims[1] + (uint64_t)iy) *
               (uint64_t)dims[0] + (uint64_t)ix;
    return true;
}

}  // namespace

extern "C" {

// Stage 1a-1c for ONE grid scale: voxel coordinates, dedup in canonical
// (ascending key) order, kept-point counts and fp32 means of all C channels.
//   cap > 0: a voxel keeps only its `cap` points of lowest original index;
//            dropped points get point_voxel = -1 (keep-first-by-index rule).
// Outputs sized for the worst case: coords [B*N,4] as (b,z,y,x), counts [B*N],
// mean [B*N,C], point_voxel [B*N] (index into the unique list, -1 if out of
// range or dropped).  Returns the number of unique voxels M.
int emc2o_voxelize(int B, int N, int C, const float* points, const float* mn, const float* vs,
                   const int* dims, int cap, int32_t* coords, int32_t* counts, float* mean,
                   int32_t* point_voxel) {
    const int64_t total = (int64_t)B * N;
    std::vector<uint64_t> keys(total);
    std::vector<char> valid(total);
    std::vector<uint64_t> uniq;
    for (int64_t i = 0; i < total; ++i) {
        int b = (int)(i / N);
        valid[i] = voxel_key(points + i * C, b, mn, vs, dims, &keys[i]);
        if (valid[i]) uniq.push_back(keys[i]);
    }
    std::sort(uniq.begin(), uniq.end());
    uniq.erase(std::unique(uniq.begin(), uniq.end()), uniq.end());
    const int M = (int)uniq.size();
    for (int m = 0; m < M; ++m) {
        uint64_t k = uniq[m];
        int ix = (int)(k % dims[0]); k /= dims[0];
        int iy = (int)(k % dims[1]); k /= dims[1];
        int iz = (int)(k % dims[2]); k /= dims[2];
        coords[4 * m + 0] = (int)k;
        coords[4 * m + 1] = iz;
        coords[4 * m + 2] = iy;
        coords[4 * m + 3] = ix;
        counts[m] = 0;
    }
    std::vector<double> sums((size_t)M * C, 0.0);
    for (int64_t i = 0; i < total; ++i) {           // ascending original index
        point_voxel[i] = -1;
        if (!valid[i]) continue;
        int m = (int)(std::lower_bound(uniq.begin(), uniq.end(), keys[i]) - uniq.begin());
        if (cap > 0 && counts[m] >= cap) continue;   // voxel already full: drop
        counts[m] += 1;
        point_voxel[i] = m;
        for (int c = 0; c < C; ++c) sums[(size_t)m * C + c] += (double)points[i * C + c];
    }
    for (int m = 0; m < M; ++m)
        for (int c = 0; c < C; ++c)
            mean[(size_t)m * C + c] = (float)(sums[(size_t)m * C + c] / (double)counts[m]);
    return M;
}

// Stage 1d: BEV pseudo-image [B, C, Gy, Gx] for the 2D expert (Sec. 3.3,
// Latency-Prioritized Expert): each pillar's mean features at (iy, ix), zero
// elsewhere.
void emc2o_bev(int B, int C, int Gy, int Gx, int M, const int32_t* coords, const float* mean,
               float* bev) {
    std::memset(bev, 0, sizeof(float) * (size_t)B * C * Gy * Gx);
    for (int m = 0; m < M; ++m) {
        int b = coords[4 * m + 0], iy = coords[4 * m + 2], ix = coords[4 * m + 3];
        for (int c = 0; c < C; ++c)
            bev[(((size_t)b * C + c) * Gy + iy) * Gx + ix] = mean[(size_t)m * C + c];
    }
}

// Stage 2a: LiDAR-to-camera projection (Sec. 3.1, "based on depth information
// it projects ..."): proj [B,K,3,4] maps (x,y,z,1) to (u*d, v*d, d).  A point
// is visible in camera k iff d > min_depth and 0 <= u < W and 0 <= v < H.
// vis_mask bit k; cam = lowest visible camera or -1; uvd of that camera, or
// (-1, -1, depth in camera 0 [0 if not finite]) when invisible.
void emc2o_project(int B, int N, int C, int K, const float* points, const float* proj, int H, int W,
                   float min_depth, float* uvd, uint8_t* vis_mask, int8_t* cam) {
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < N; ++i) {
            const int64_t g = (int64_t)b * N + i;
            const float x = points[g * C + 0], y = points[g * C + 1], z = points[g * C + 2];
            unsigned mask = 0;
            int best = -1;
            float bu = -1.0f, bv = -1.0f, bd = 0.0f, d0 = 0.0f;
            for (int k = 0; k < K; ++k) {
                const float* P = proj + ((size_t)b * K + k) * 12;
                float t[3];
                for (int r = 0; r < 3; ++r)
                    t[r] = std::fmaf(P[4 * r + 0], x,
                                     std::fmaf(P[4 * r + 1], y, std::fmaf(P[4 * r + 2], z, P[4 * r + 3])));
                if (k == 0) d0 = t[2];
                if (!(t[2] > min_depth)) continue;
                float u = t[0] / t[2], v = t[1] / t[2];
                bool vis = (u >= 0.0f) && (u < (float)W) && (v >= 0.0f) && (v < (float)H);
                if (!vis) continue;
                mask |= 1u << k;
                if (best < 0) { best = k; bu = u; bv = v; bd = t[2]; }
            }
            if (best < 0) bd = std::isfinite(d0) ? d0 : 0.0f;
            uvd[3 * g + 0] = bu; uvd[3 * g + 1] = bv; uvd[3 * g + 2] = bd;
            vis_mask[g] = (uint8_t)mask;
            cam[g] = (int8_t)best;
        }
}

// Stage 2b: bilinear gather from the chosen camera's channels-last feature map
// feat [B,K,Hf,Wf,Cf].  Texel (j,i) is the sample at pixel (j*s, i*s); taps
// are edge-clamped; points with cam = -1 get an all-zero row (Fig. 5: no match
// -> zero-filled features).  The blend is evaluated in double and rounded once.
void emc2o_gather(int B, int N, int K, int Hf, int Wf, int Cf, int stride, float offset, const float* uvd,
                  const int8_t* cam, const float* feat, float* gathered) {
    // `offset` is the pixel position of texel 0 (0 for a plain strided map; (p - 1) / 2 * s for a
    // map that was average-pooled p x p, whose texels sit at the centres of their windows).
    const double inv = 1.0 / (double)stride;
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < N; ++i) {
            const int64_t g = (int64_t)b * N + i;
            float* out = gathered + g * Cf;
            if (cam[g] < 0) {
                for (int c = 0; c < Cf; ++c) out[c] = 0.0f;
                continue;
            }
            // The subtraction is done in fp32 (one rounding), as the pixel coordinates are fp32.
            double fx = (double)(uvd[3 * g + 0] - offset) * inv, fy = (double)(uvd[3 * g + 1] - offset) * inv;
            int x0 = (int)std::floor(fx), y0 = (int)std::floor(fy);
            double wx = fx - x0, wy = fy - y0;
            int x1 = std::min(x0 + 1, Wf - 1), y1 = std::min(y0 + 1, Hf - 1);
            x0 = std::min(x0, Wf - 1);
            y0 = std::min(y0, Hf - 1);
            x0 = std::max(x0, 0); x1 = std::max(x1, 0);     // left of texel 0: clamp to the edge as well
            y0 = std::max(y0, 0); y1 = std::max(y1, 0);
            const float* base = feat + ((size_t)b * K + cam[g]) * Hf * Wf * Cf;
            const float* f00 = base + ((size_t)y0 * Wf + x0) * Cf;
            const float* f01 = base + ((size_t)y0 * Wf + x1) * Cf;
            const float* f10 = base + ((size_t)y1 * Wf + x0) * Cf;
            const float* f11 = base + ((size_t)y1 * Wf + x1) * Cf;
            for (int c = 0; c < Cf; ++c) {
                double top = (1.0 - wx) * f00[c] + wx * f01[c];
                double bot = (1.0 - wx) * f10[c] + wx * f11[c];
                out[c] = (float)((1.0 - wy) * top + wy * bot);
            }
        }
}

// Multiscale Pooling of the image features (Sec. 3.5: image features are pooled, with a
// user-chosen pooling size, before they are fused with LiDAR features, to relieve memory).
// feat [B,K,Hf,Wf,Cf] channels-last -> pooled [B,K,ceil(Hf/p),ceil(Wf/p),Cf]: the mean over each
// p x p window of texels; windows at the right / bottom edge hold fewer texels and average over
// those they hold.
void emc2o_pool(int B, int K, int Hf, int Wf, int Cf, int p, const float* feat, float* pooled) {
    const int Hp = (Hf + p - 1) / p, Wp = (Wf + p - 1) / p;
    for (int m = 0; m < B * K; ++m)
        for (int J = 0; J < Hp; ++J)
            for (int I = 0; I < Wp; ++I)
                for (int c = 0; c < Cf; ++c) {
                    double sum = 0.0;
                    int n = 0;
                    for (int j = J * p; j < std::min(Hf, J * p + p); ++j)
                        for (int i = I * p; i < std::min(Wf, I * p + p); ++i) {
                            sum += (double)feat[(((size_t)m * Hf + j) * Wf + i) * Cf + c];
                            n += 1;
                        }
                    pooled[(((size_t)m * Hp + J) * Wp + I) * Cf + c] = (float)(sum / n);
                }
}

// Stage 3: per-point routing (Sec. 3.2: near is "< D", far is ">= D").  Planar
// range squared r2 = fma(x, x, y*y) in fp32 is compared with squared
// thresholds t*t (fp32); the distance bucket is the number of thresholds
// reached; expert = lut[visible][bucket], lut is [2][8].
void emc2o_route(int B, int N, int C, const float* points, const uint8_t* vis_mask, int T,
                 const float* thresholds, const uint8_t* lut, uint8_t* expert) {
    float t2[8];
    for (int t = 0; t < T; ++t) t2[t] = thresholds[t] * thresholds[t];
    for (int64_t g = 0; g < (int64_t)B * N; ++g) {
        float x = points[g * C + 0], y = points[g * C + 1];
        float r2 = std::fmaf(x, x, y * y);
        int bucket = 0;
        for (int t = 0; t < T; ++t) bucket += (r2 >= t2[t]) ? 1 : 0;
        expert[g] = lut[(vis_mask[g] != 0 ? 8 : 0) + bucket];
    }
}

// Stage 4: stable counting-sort partition per frame (offsets are the exclusive
// prefix sum of the per-expert counts, Sec. 3.6).  offsets [B,E+1],
// perm [B,N] with out[j] = in[perm[j]] (frame-local indices), then the point
// and feature rows are copied in that order.
void emc2o_dispatch(int B, int N, int C, int Cf, int E, const uint8_t* expert, const float* points,
                    const float* gathered, int32_t* offsets, int32_t* perm, float* points_out,
                    float* feat_out) {
    for (int b = 0; b < B; ++b) {
        const uint8_t* ex = expert + (size_t)b * N;
        int32_t* off = offsets + (size_t)b * (E + 1);
        std::vector<int32_t> cnt(E, 0);
        for (int i = 0; i < N; ++i) cnt[ex[i]] += 1;
        off[0] = 0;
        for (int e = 0; e < E; ++e) off[e + 1] = off[e] + cnt[e];
        std::vector<int32_t> cursor(off, off + E);
        for (int i = 0; i < N; ++i) perm[(size_t)b * N + cursor[ex[i]]++] = i;
        for (int j = 0; j < N; ++j) {
            const int64_t src = (int64_t)b * N + perm[(size_t)b * N + j], dst = (int64_t)b * N + j;
            std::memcpy(points_out + dst * C, points + src * C, sizeof(float) * C);
            std::memcpy(feat_out + dst * Cf, gathered + src * Cf, sizeof(float) * Cf);
        }
    }
}

}  // extern "C"

// Scene-level choice of the Scenario-Adaptive Dispatcher (Sec. 3.2): a scene goes to the most
// demanding expert that any of its objects asks for (close-and-distinct scenes to the
// latency-prioritised expert, scenes with some harder object to the next one, and so on).  Per
// point, that is the expert of highest priority among those that own at least `min_points`
// points of the frame; ties go to the lowest expert id; -1 if no expert qualifies.
// offsets [B, E+1] as written by the dispatch; priority [E]; scene_expert [B].
extern "C" void emc2o_scene_route(int B, int E, const int32_t* offsets, const uint8_t* priority, int min_points,
                                  int32_t* scene_expert) {
    if (min_points < 1) min_points = 1;
    for (int b = 0; b < B; ++b) {
        const int32_t* off = offsets + (size_t)b * (E + 1);
        int best = -1;
        for (int e = 0; e < E; ++e) {
            const int count = off[e + 1] - off[e];
            if (count < min_points) continue;
            if (best < 0 || priority[e] > priority[best]) best = e;
        }
        scene_expert[b] = best;
    }
}

// Fusion by voxel (Fig. 5): the image features of the pixels that share a voxel's 3-D coordinate
// go with that voxel; voxels without such pixels get zero-filled features.  Here the pixels with
// a 3-D coordinate are the projected LiDAR points, so voxel m receives the mean of the gathered
// rows of its kept points that some camera sees (vis_mask != 0), and a zero row if it has none.
// point_voxel [B*N] (row of the point's voxel, -1 if none), vis_mask [B*N], gathered [B*N, Cf] ->
// vox_img [M, Cf], vox_img_count [M] (points averaged).
extern "C" void emc2o_voxel_image(long long total, int M, int Cf, const int32_t* point_voxel, const uint8_t* vis_mask,
                                  const float* gathered, float* vox_img, int32_t* vox_img_count) {
    std::vector<double> sums((size_t)M * Cf, 0.0);
    for (int m = 0; m < M; ++m) vox_img_count[m] = 0;
    for (long long i = 0; i < total; ++i) {
        const int m = point_voxel[i];
        if (m < 0 || m >= M || vis_mask[i] == 0) continue;
        vox_img_count[m] += 1;
        for (int c = 0; c < Cf; ++c) sums[(size_t)m * Cf + c] += (double)gathered[i * Cf + c];
    }
    for (int m = 0; m < M; ++m)
        for (int c = 0; c < Cf; ++c)
            vox_img[(size_t)m * Cf + c] =
                vox_img_count[m] ? (float)(sums[(size_t)m * Cf + c] / (double)vox_img_count[m]) : 0.0f;
}

// Occlusion test for the "occluded / out-of-view" bucket.  The paper names occlusion as a cause of
// missing LiDAR detail (Sec. 3.2, case 3) but gives no test; this is the usual depth-buffer one.
// Every camera image is cut into cells of `cell` x `cell` pixels (cell a power of two).  For each
// camera that sees a point (bit k of vis_mask), the point falls into cell (floor(v/cell),
// floor(u/cell)) with depth d, both from the same fp32 projection as emc2o_project.  zbuf holds the
// smallest depth per cell.  The point is occluded in camera k iff d > zbuf + margin (fp32 add,
// fp32 compare).  occ_mask bit k = occluded in camera k; clear_mask = vis_mask & ~occ_mask.
// zbuf [B,K,Hz,Wz] with Hz = ceil(H/cell), Wz = ceil(W/cell); +infinity where no point falls.
extern "C" void emc2o_occlusion(int B, int N, int C, int K, const float* points, const float* proj, int H, int W,
                                const uint8_t* vis_mask, int cell, float margin, float* zbuf, uint8_t* occ_mask,
                                uint8_t* clear_mask) {
    const int Hz = (H + cell - 1) / cell, Wz = (W + cell - 1) / cell;
    const float inv = 1.0f / (float)cell;
    const size_t nz = (size_t)B * K * Hz * Wz;
    for (size_t i = 0; i < nz; ++i) zbuf[i] = INFINITY;
    std::vector<float> depth((size_t)B * N * K, 0.0f);
    std::vector<int> where((size_t)B * N * K, -1);
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < N; ++i) {
            const int64_t g = (int64_t)b * N + i;
            const float x = points[g * C + 0], y = points[g * C + 1], z = points[g * C + 2];
            for (int k = 0; k < K; ++k) {
                if (!((vis_mask[g] >> k) & 1)) continue;
                const float* P = proj + ((size_t)b * K + k) * 12;
                float t[3];
                for (int r = 0; r < 3; ++r)
                    t[r] = std::fmaf(P[4 * r + 0], x,
                                     std::fmaf(P[4 * r + 1], y, std::fmaf(P[4 * r + 2], z, P[4 * r + 3])));
                const float u = t[0] / t[2], v = t[1] / t[2];
                const int cx = std::min((int)std::floor(u * inv), Wz - 1), cy = std::min((int)std::floor(v * inv), Hz - 1);
                const size_t c = (((size_t)b * K + k) * Hz + cy) * Wz + cx;
                depth[g * K + k] = t[2];
                where[g * K + k] = (int)c;
                zbuf[c] = std::min(zbuf[c], t[2]);
            }
        }
    for (int64_t g = 0; g < (int64_t)B * N; ++g) {
        unsigned occ = 0;
        for (int k = 0; k < K; ++k) {
            const int c = where[g * K + k];
            if (c < 0) continue;
            const float lim = zbuf[c] + margin;
            if (depth[g * K + k] > lim) occ |= 1u << k;
        }
        occ_mask[g] = (uint8_t)occ;
        clear_mask[g] = (uint8_t)(vis_mask[g] & ~occ);
    }
}

// Layout change for callers whose image branch emits planar maps: [B,K,Cf,Hf,Wf] -> the
// channels-last [B,K,Hf,Wf,Cf] the gather reads.  A pure copy.
extern "C" void emc2o_channels_last(int maps, int Cf, int Hf, int Wf, const float* planar, float* last) {
    for (int m = 0; m < maps; ++m)
        for (int c = 0; c < Cf; ++c)
            for (int j = 0; j < Hf; ++j)
                for (int i = 0; i < Wf; ++i)
                    last[(((size_t)m * Hf + j) * Wf + i) * Cf + c] = planar[(((size_t)m * Cf + c) * Hf + j) * Wf + i];
}

// Rulebook of a 3 x 3 x 3 submanifold sparse convolution over a voxel list (the index structure
// of the 3D sparse convolution of Sec. 3.5, which runs on the non-empty voxels only; Sec. 3.6
// replaces its index search by prefix sums).  The paper gives neither the kernel size nor the
// layout: this is the usual one.  Kernel offset k = (dz+1)*9 + (dy+1)*3 + (dx+1) with dz, dy, dx
// in {-1, 0, 1}.  For every k, in ascending order of the output voxel m: if a voxel n of the same
// frame sits at coords[m] + (dz, dy, dx), the pair (in = n, out = m) is appended.
// coords [M, 4] rows (b, z, y, x), all different -> offsets [28] (pairs before offset k; [27] =
// all pairs), rule_in / rule_out [<= 27 * M].  Returns the number of pairs.
extern "C" long long emc2o_rulebook(int M, const int32_t* coords, int32_t* offsets, int32_t* rule_in,
                                    int32_t* rule_out) {
    std::map<std::array<int32_t, 4>, int32_t> where;
    for (int m = 0; m < M; ++m)
        where[{coords[4 * m], coords[4 * m + 1], coords[4 * m + 2], coords[4 * m + 3]}] = m;
    long long pairs = 0;
    int k = 0;
    for (int dz = -1; dz <= 1; ++dz)
        for (int dy = -1; dy <= 1; ++dy)
            for (int dx = -1; dx <= 1; ++dx, ++k) {
                offsets[k] = (int32_t)pairs;
                for (int m = 0; m < M; ++m) {
                    const int32_t* c = coords + 4 * m;
                    auto it = where.find({c[0], c[1] + dz, c[2] + dy, c[3] + dx});
                    if (it == where.end()) continue;
                    rule_in[pairs] = it->second;
                    rule_out[pairs] = m;
                    pairs += 1;
                }
            }
    offsets[27] = (int32_t)pairs;
    return pairs;
}
