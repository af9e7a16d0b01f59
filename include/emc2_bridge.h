/*
 * emc2_bridge.h -- C ABI of the B200 (sm_100a) multimodal data bridge and dispatch.
 *
 * The library implements, as CUDA kernels, the non-learned work that runs on
 * every frame before any expert model of EMC2 (arXiv 2507.04123):
 *   - the Adaptive Multimodal Data Bridge's preprocessing (Sec. 3.1): LiDAR
 *     voxelization at two grid scales with per-voxel counts and mean features,
 *     the BEV pseudo-image the 2D expert consumes (Sec. 3.3), LiDAR-to-camera
 *     projection and sampling of image features, with zero rows where a point
 *     has no pixel (Fig. 5);
 *   - the Scenario-Adaptive Dispatcher's distance rule (Sec. 3.2: "close" is
 *     < D, "distant" is >= D), applied per point together with visibility;
 *   - the dispatch of points and features into contiguous per-expert buffers,
 *     indexed by prefix sums (Sec. 3.6).
 *
 * General rules
 *   - Every pointer named d_* is DEVICE memory on the handle's device, owned by
 *     the caller, contiguous, row-major and 16-byte aligned.  Pointers named
 *     h_* or without prefix are HOST memory.  The library never frees or keeps
 *     a caller pointer after the call has been enqueued.
 *   - Every call that takes `cuda_stream` (a cudaStream_t passed as void*,
 *     NULL = legacy default stream) only enqueues kernels.  These calls do not
 *     allocate, do not synchronise and do not touch the host except to return.
 *     Some kernels are cooperative launches (grid-wide barrier), which the
 *     device must support; emc2_bridge_create() fails otherwise.  The calls
 *     that take a handle and a stream can therefore be captured into a CUDA
 *     graph and replayed (emc2_bridge_status synchronises and cannot).
 *   - One handle serves one device and one stream at a time; it is not
 *     thread-safe.  Calls on the same handle must be ordered on the stream.
 *   - Errors are returned as negative emc2_status_t values.  Errors the host
 *     can see (null or misaligned pointer, sizes over the configured maxima)
 *     return at once and enqueue nothing.  Errors only the device can see
 *     (more unique voxels than `capacity`) set a sticky status word that
 *     emc2_bridge_status() reads.  Nothing aborts, traps or prints.
 *   - There is no CPU fallback: without a CUDA device create() fails.
 */
#ifndef EMC2_BRIDGE_H
#define EMC2_BRIDGE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    EMC2_OK = 0,
    EMC2_ERR_INVALID_ARG = -1, /* null/misaligned pointer, B or N outside the configured maxima; from
                                  emc2_bridge_status: a voxel list that is not one of its grid */
    EMC2_ERR_BAD_CONFIG = -2,  /* emc2_config_t rejected by emc2_bridge_create */
    EMC2_ERR_CUDA = -3,        /* a CUDA runtime call failed; see emc2_bridge_last_cuda_error */
    EMC2_ERR_CAPACITY = -4,    /* more unique voxels than capacity[s] (device-detected, sticky) */
    EMC2_ERR_TIMEOUT = -5,     /* reserved: a bounded device-side wait gave up.  No kernel of this library
                                  spins on another CTA (the only grid-wide waits are the barriers of
                                  cooperative launches), so it is never returned at present */
    EMC2_ERR_INTERNAL = -6,    /* from emc2_bridge_status: a call found the handle's scratch in use (two
                                  calls on one handle at once); that call's voxel outputs are void and the
                                  handle should be destroyed */
    EMC2_ERR_TOO_LARGE = -7    /* the call needs more scratch than a fixed-size scratch area holds */
} emc2_status_t;

#define EMC2_MAX_CAMERAS 8
#define EMC2_MAX_THRESHOLDS 7
#define EMC2_MAX_EXPERTS 16
#define EMC2_MAX_BATCH 32

typedef struct emc2_bridge emc2_bridge_t; /* opaque; owns scratch memory and the device status word */

/* One voxel grid (Sec. 3.1 "multi-scale preprocessing").  A point p lies in cell
 * i_d = floor((p_d - min[d]) / voxel[d]) (fp32 subtract, fp32 IEEE divide) and is inside the
 * grid iff 0 <= i_d < dims[d] on all three axes; non-finite coordinates are outside. */
typedef struct {
    float min[3];       /* lower corner (x, y, z), metres */
    float voxel[3];     /* cell size (x, y, z), metres, > 0 */
    int32_t dims[3];    /* cells along (x, y, z) = (Gx, Gy, Gz) */
    int32_t max_points; /* per-voxel cap; 0 = none.  With a cap a voxel keeps its max_points
                           points of lowest index within the batch; the rest are dropped. */
} emc2_grid_t;

typedef struct {
    int32_t device;       /* CUDA device ordinal */
    int32_t max_batch;    /* largest B of any call, 1..EMC2_MAX_BATCH */
    int32_t max_points;   /* largest N (points per frame) of any call */
    int32_t point_floats; /* C: floats per point, 4 (x,y,z,intensity) or 5 (+ time lag) */
    emc2_grid_t grid[2];  /* [0] fine voxels, [1] pillars (dims[2] == 1) */
    int32_t num_cameras;  /* K, 1..EMC2_MAX_CAMERAS */
    int32_t img_h, img_w; /* image size in pixels */
    int32_t feat_h, feat_w, feat_c; /* feature map size; feat_c a multiple of 4 */
    int32_t feat_stride;  /* s: texel (j, i) is the sample at pixel (j*s, i*s); a power of two */
    float min_depth;      /* a point is visible only if its depth is > min_depth */
    int32_t num_thresholds;                /* T, 0..EMC2_MAX_THRESHOLDS */
    float thresholds[EMC2_MAX_THRESHOLDS]; /* ascending planar ranges in metres */
    int32_t num_experts;                   /* E, 1..EMC2_MAX_EXPERTS */
    uint8_t lut[2][8]; /* expert = lut[visible ? 1 : 0][number of thresholds reached]; < E */
    float feat_offset; /* pixel position of texel 0 along both axes: texel (j, i) is the sample at pixel
                          (feat_offset + j*s, feat_offset + i*s).  0 for a plain strided map; (p-1)/2 * s0
                          for a map that emc2_pool_features pooled p x p from stride s0 (then s = p*s0).
                          Finite, >= 0. */
} emc2_config_t;

/* Validates the configuration, selects the device and allocates all scratch memory the stage
 * calls will ever need for (max_batch, max_points).  Returns EMC2_ERR_BAD_CONFIG for an
 * unusable configuration (zero voxel size, more than 2^32 - 1 cells per batch,
 * feat_c not a multiple of 4, stride not a power of two,
 * lut entry >= num_experts, ...), EMC2_ERR_CUDA if the device or memory is unavailable. */
int emc2_bridge_create(const emc2_config_t* config, emc2_bridge_t** out);

/* Stage 1 (Sec. 3.1; BEV for the 2D expert of Sec. 3.3).  For each scale s in {0, 1}:
 *   d_coords[s]      int32 [capacity[s], 4]  unique voxels as (b, z, y, x), ascending in that order
 *   d_counts[s]      int32 [capacity[s]]     points kept in the voxel (<= max_points if capped)
 *   d_mean[s]        float [capacity[s], C]  mean of the kept points over all C channels
 *   d_point_voxel[s] int32 [B, N] or NULL    row of the point's voxel; -1 if outside the grid or
 *                                            dropped by the cap
 *   d_num_voxels     int32 [2]               number of unique voxels found per scale (true count
 *                                            even when it exceeds capacity[s])
 *   d_bev            float [B, C, Gy, Gx] of grid[1], or NULL: pillar means at (iy, ix), else 0
 * d_points is float [B, N, C].  Rows past num_voxels are left untouched.  All integer outputs
 * (coordinates, counts, point rows, the number of voxels) are the same on every run; the means
 * and the BEV image are sums of fp32 reductions whose order is not fixed, so they are
 * reproducible to the comparison tolerance (1e-4 + 1e-5 |x|), not bit for bit.  The same holds
 * for the rows of emc2_voxel_image and its variants.  If a scale finds more
 * voxels than capacity[s], rows past capacity are not written and EMC2_ERR_CAPACITY becomes
 * sticky.  d_coords, d_counts, d_mean and capacity are HOST arrays of two entries. */
int emc2_voxelize(emc2_bridge_t* bridge, int32_t B, int32_t N, const float* d_points,
                  int32_t* const d_coords[2], int32_t* const d_counts[2], float* const d_mean[2],
                  int32_t* const d_point_voxel[2], const int32_t capacity[2], int32_t* d_num_voxels,
                  float* d_bev, void* cuda_stream);

/* Stage 2 (Sec. 3.1 projection "based on depth information"; Fig. 5 zero fill).
 *   d_proj      float [B, K, 3, 4]  row-major; maps LiDAR-frame (x, y, z, 1) to (u*d, v*d, d)
 *   d_feat      float [B, K, Hf, Wf, Cf]  channels-last feature maps
 *   d_uvd       float [B, N, 3]   (u, v, depth) in the lowest-index camera that sees the point,
 *                                 or (-1, -1, depth in camera 0 [0 if not finite]) if none does
 *   d_vis_mask  uint8 [B, N]      bit k set iff depth_k > min_depth, 0 <= u < W and 0 <= v < H
 *   d_cam       int8  [B, N]      that camera, or -1
 *   d_gathered  float [B, N, Cf]  bilinear sample at ((u - feat_offset)/s, (v - feat_offset)/s), taps
 *                                 clamped to the map edge;
 *                                 all zeros for points no camera sees */
int emc2_project_gather(emc2_bridge_t* bridge, int32_t B, int32_t N, const float* d_points,
                        const float* d_proj, const float* d_feat, float* d_uvd, uint8_t* d_vis_mask,
                        int8_t* d_cam, float* d_gathered, void* cuda_stream);

/* Stages 3 and 4 (Sec. 3.2 distance rule; Sec. 3.6 prefix sums).  Per frame b:
 *   d_expert      uint8 [B, N]     lut[vis_mask != 0][#{t : x*x + y*y >= thresholds[t]^2}]
 *   d_offsets     int32 [B, E+1]   exclusive prefix sum of per-expert counts; offsets[b][E] = N
 *   d_perm        int32 [B, N]     frame-local source index of output row j (stable: ascending
 *                                  inside each expert's segment)
 *   d_points_out  float [B, N, C]  points[b][perm[b][j]]
 *   d_feat_out    float [B, N, Cf] gathered[b][perm[b][j]]
 * d_vis_mask and d_gathered are the outputs of emc2_project_gather (or any buffers of that
 * shape).  Outputs must not alias inputs. */
int emc2_route_dispatch(emc2_bridge_t* bridge, int32_t B, int32_t N, const float* d_points,
                        const uint8_t* d_vis_mask, const float* d_gathered, uint8_t* d_expert,
                        int32_t* d_offsets, int32_t* d_perm, float* d_points_out, float* d_feat_out,
                        void* cuda_stream);

/* The whole bridge in one call (all four stages; Sec. 3.1 - 3.2, with the overlap of independent
 * work that Sec. 3.6 asks of the system).  Arguments, outputs, layouts and errors are exactly those
 * of emc2_voxelize, emc2_project_gather and emc2_route_dispatch called in that order with the same
 * buffers.  Stages 2 - 4 run as one pass: the expert id is computed beside the projection, and
 * every feature row is blended once and stored both at its row of d_gathered and at its slot of
 * d_feat_out, so the rows are not read back.  The pass over the points that
 * projects and routes them also marks their voxel cells, so stage 1 reads the points once less.
 * The rest of stage 1 does not depend on stages 2 - 4, so the library runs it on a stream of its own
 * (created with the handle, highest priority) beside them: it starts once that first pass, and with it
 * the work already queued on `cuda_stream`, has finished, and `cuda_stream` waits for it before the
 * call's work counts as complete.  Seen from
 * `cuda_stream` the call therefore behaves like the three calls, only shorter.  No allocation,
 * no host synchronisation.  d_gathered may be NULL for a caller who consumes only the dispatched
 * rows (d_feat_out with d_perm): the rows in point order are then not stored, which saves their
 * 4 * Cf bytes per point of memory traffic. */
int emc2_bridge_run(emc2_bridge_t* bridge, int32_t B, int32_t N, const float* d_points, const float* d_proj,
                    const float* d_feat, int32_t* const d_coords[2], int32_t* const d_counts[2],
                    float* const d_mean[2], int32_t* const d_point_voxel[2], const int32_t capacity[2],
                    int32_t* d_num_voxels, float* d_bev, float* d_uvd, uint8_t* d_vis_mask, int8_t* d_cam,
                    float* d_gathered, uint8_t* d_expert, int32_t* d_offsets, int32_t* d_perm,
                    float* d_points_out, float* d_feat_out, void* cuda_stream);

/* emc2_bridge_run for a caller whose frame lives in HOST memory (the sensor side of Sec. 3.1: LiDAR
 * points, calibration and image features arrive on the host): enqueues, on `cuda_stream`, the copies
 * of h_points [B, N, C], h_proj [B, K, 3, 4] and h_feat [B, K, Hf, Wf, Cf] into the caller's device
 * buffers d_points, d_proj, d_feat, then emc2_bridge_run on them with the same outputs, then the
 * copies of d_offsets [B, E+1] and d_num_voxels [2] into h_offsets and h_num_voxels (either may be
 * NULL: not copied).  Nothing is synchronised: the host buffers must stay valid and unchanged until
 * the stream has passed the call; the copies are asynchronous only for page-locked host memory
 * (which stream capture requires).  A
 * caller who alternates between two handles, streams and buffer sets overlaps one frame's copies with
 * the other's kernels. */
int emc2_bridge_run_host(emc2_bridge_t* bridge, int32_t B, int32_t N, const float* h_points, const float* h_proj,
                         const float* h_feat, float* d_points, float* d_proj, float* d_feat,
                         int32_t* const d_coords[2], int32_t* const d_counts[2], float* const d_mean[2],
                         int32_t* const d_point_voxel[2], const int32_t capacity[2], int32_t* d_num_voxels,
                         float* d_bev, float* d_uvd, uint8_t* d_vis_mask, int8_t* d_cam, float* d_gathered,
                         uint8_t* d_expert, int32_t* d_offsets, int32_t* d_perm, float* d_points_out,
                         float* d_feat_out, int32_t* h_offsets, int32_t* h_num_voxels, void* cuda_stream);

/* Layout change for callers whose image branch (a ResNet in Sec. 3.1) emits planar maps: copies
 * d_planar float [B, K, Cf, Hf, Wf] into d_feat float [B, K, Hf, Wf, Cf], the channels-last layout
 * the gather reads (one tap = one contiguous row).  The handle's K, Hf, Wf, Cf apply; the two
 * buffers must not overlap. */
int emc2_features_channels_last(emc2_bridge_t* bridge, int32_t B, const float* d_planar, float* d_feat,
                                void* cuda_stream);

/* Multiscale Pooling of the image features (Sec. 3.5: image features are pooled, with a pooling size
 * the user chooses, before they are fused with LiDAR features, to relieve memory).
 *   d_feat    float [B, K, Hf, Wf, Cf]                    the handle's feature-map shape
 *   d_pooled  float [B, K, ceil(Hf/p), ceil(Wf/p), Cf]    mean over each p x p window of texels; windows
 *                                                         at the right / bottom edge average over the
 *                                                         texels they hold
 * p >= 1 (1 copies).  To sample the pooled maps, use a handle whose configuration has
 * feat_h = ceil(Hf/p), feat_w = ceil(Wf/p), feat_stride = p * s (p a power of two) and
 * feat_offset = (p - 1) / 2 * s, so that each pooled texel sits at the centre of its window. */
int emc2_pool_features(emc2_bridge_t* bridge, int32_t B, int32_t p, const float* d_feat, float* d_pooled,
                       void* cuda_stream);

/* Rulebook of a 3 x 3 x 3 submanifold sparse convolution over one scale's voxel list: the index
 * structure of the 3D sparse convolution that consumes the list (Sec. 3.5), built with prefix sums
 * instead of an index search (Sec. 3.6).  The paper states neither kernel size nor layout; this is
 * the usual one.  Kernel offset k = (dz+1)*9 + (dy+1)*3 + (dx+1), dz, dy, dx in {-1, 0, 1}.
 *   d_rule_offsets  int32 [28]             pairs before offset k; [27] = all pairs (true count even
 *                                          when it exceeds pair_capacity)
 *   d_rule_in/out   int32 [pair_capacity]  for every k, in ascending out: the pairs (in = n, out = m)
 *                                          with coords[n] = coords[m] + (0, dz, dy, dx), same frame
 * d_coords int32 [capacity, 4] and d_num_voxels (DEVICE int32, the scale's entry) are emc2_voxelize's
 * outputs for grid[scale]: rows (b, z, y, x) inside the grid, all different, in ascending order;
 * min(*d_num_voxels, capacity) rows are used, capacity <= max_batch * max_points.  A list that
 * breaks these rules makes EMC2_ERR_INVALID_ARG sticky (device-detected; the outputs are then
 * undefined but in bounds).  27 * capacity pairs always suffice; with fewer, pairs past
 * pair_capacity are not written and EMC2_ERR_CAPACITY becomes sticky.  Enqueues five kernels; uses
 * the scale's handle scratch, so calls on one handle must be ordered. */
int emc2_rulebook(emc2_bridge_t* bridge, int32_t scale, int32_t capacity, const int32_t* d_coords,
                  const int32_t* d_num_voxels, int32_t* d_rule_offsets, int32_t* d_rule_in, int32_t* d_rule_out,
                  int64_t pair_capacity, void* cuda_stream);

/* Fusion by voxel (Fig. 5: image features of the pixels that share a voxel's 3-D coordinate go with
 * that voxel; voxels without such pixels get zero-filled features).  The pixels with a 3-D coordinate
 * are the projected points, so for one voxel scale:
 *   d_vox_img        float [capacity, Cf]  row m = mean of d_gathered over the points i with
 *                                          d_point_voxel[i] == m and d_vis_mask[i] != 0; zeros if none
 *   d_vox_img_count  int32 [capacity]      number of points averaged
 * Inputs are outputs of the earlier stages for the SAME scale and batch: d_point_voxel [B, N],
 * d_counts [capacity], d_num_voxels -> the scale's entry (DEVICE int32), d_vis_mask [B, N],
 * d_gathered [B, N, Cf].  Rows past min(*d_num_voxels, capacity) are left untouched.  Concatenating
 * [d_mean row | d_vox_img row] gives the fused voxel feature; the library leaves that to the consumer.
 * Enqueues three kernels on `cuda_stream`; uses handle scratch, so calls on one handle must be
 * ordered.  d_counts that add up to more than B * N (not this batch's counts) make
 * EMC2_ERR_INVALID_ARG sticky and nothing is written. */
int emc2_voxel_image(emc2_bridge_t* bridge, int32_t B, int32_t N, int32_t capacity, const int32_t* d_point_voxel,
                     const int32_t* d_counts, const int32_t* d_num_voxels, const uint8_t* d_vis_mask,
                     const float* d_gathered, float* d_vox_img, int32_t* d_vox_img_count, void* cuda_stream);

/* Fusion by voxel straight from the feature maps (Fig. 5 again; this is the per-voxel form of the
 * bridge's image branch: the per-point rows of emc2_project_gather are neither written nor read).
 * Outputs as emc2_voxel_image.  Instead of the gathered rows and the visibility mask the call takes
 * d_uvd float [B, N, 3] and d_cam int8 [B, N] of the projection stage and the feature maps d_feat
 * float [B, K, Hf, Wf, Cf]; a point counts iff d_cam >= 0, and its row is the bilinear blend the
 * gather stage would have produced.  Same scratch, same ordering rule as emc2_voxel_image. */
int emc2_voxel_image_sampled(emc2_bridge_t* bridge, int32_t B, int32_t N, int32_t capacity,
                             const int32_t* d_point_voxel, const int32_t* d_counts, const int32_t* d_num_voxels,
                             const float* d_uvd, const int8_t* d_cam, const float* d_feat, float* d_vox_img,
                             int32_t* d_vox_img_count, void* cuda_stream);

/* Multiscale Pooling folded into the fusion by voxel (Sec. 3.5 pools the image features before they
 * are fused, to relieve memory; Fig. 5 fuses by voxel): the result of emc2_pool_features(p) followed by
 * emc2_voxel_image_sampled on the pooled maps, without the pooled maps ever being written or read.
 * d_feat are the handle's UNPOOLED maps [B, K, Hf, Wf, Cf]; p is the pooling size, a power of two
 * (1 = emc2_voxel_image_sampled).  Every tap of the bilinear blend is the mean of the p x p window of
 * texels that the pooled texel stands for (ragged windows at the right / bottom edge average over the
 * texels they hold); the pooled texels sit at the centres of their windows, as in emc2_pool_features.
 * d_uvd and d_cam come from a projection with the same images (they do not depend on the maps).
 * Other arguments, outputs, scratch and ordering rule as emc2_voxel_image_sampled. */
int emc2_voxel_image_pooled(emc2_bridge_t* bridge, int32_t B, int32_t N, int32_t capacity,
                            const int32_t* d_point_voxel, const int32_t* d_counts, const int32_t* d_num_voxels,
                            const float* d_uvd, const int8_t* d_cam, const float* d_feat, int32_t p,
                            float* d_vox_img, int32_t* d_vox_img_count, void* cuda_stream);

/* Occlusion test for the "occluded / out-of-view" bucket of the dispatcher (Sec. 3.2 names occlusion
 * among the causes of missing LiDAR detail; the paper gives no test, this is a depth buffer).  Every
 * camera image is cut into cells of cell x cell pixels (cell a power of two).  For each camera k that
 * sees a point (bit k of d_vis_mask) the point falls into cell (floor(v/cell), floor(u/cell)) with its
 * depth d; the buffer keeps the smallest depth per cell; the point is occluded in camera k iff
 * d > buffer + margin (fp32).
 *   d_vis_mask    uint8 [B, N]            from emc2_project_gather / emc2_bridge_run (same points, proj)
 *   d_zbuf        float [B, K, Hz, Wz]    Hz = ceil(H/cell), Wz = ceil(W/cell); written: the smallest
 *                                         depth per cell, +infinity where no point falls
 *   d_occ_mask    uint8 [B, N]            bit k: occluded in camera k
 *   d_clear_mask  uint8 [B, N]            d_vis_mask & ~d_occ_mask: pass this to emc2_route_dispatch in
 *                                         place of d_vis_mask to route occluded points as not visible
 * margin >= 0, metres.  Enqueues three kernels on `cuda_stream`. */
int emc2_occlusion(emc2_bridge_t* bridge, int32_t B, int32_t N, const float* d_points, const float* d_proj,
                   const uint8_t* d_vis_mask, int32_t cell, float margin, float* d_zbuf, uint8_t* d_occ_mask,
                   uint8_t* d_clear_mask, void* cuda_stream);

/* Scene-level choice of the Scenario-Adaptive Dispatcher (Sec. 3.2): a scene is served by the most
 * demanding expert that any of its objects asks for.  Per point: for every frame b the expert of
 * highest priority[e] among the experts that own at least max(1, min_points) points of the frame
 * (their counts are offsets[b][e+1] - offsets[b][e]); ties go to the lowest expert id; -1 if no
 * expert qualifies.
 *   d_offsets       int32 [B, E+1]  as written by emc2_route_dispatch / emc2_bridge_run
 *   priority        uint8 [E]       HOST array, larger = more demanding expert
 *   d_scene_expert  int32 [B]       output
 * Enqueues one small kernel on `cuda_stream`. */
int emc2_scene_route(emc2_bridge_t* bridge, int32_t B, const int32_t* d_offsets, const uint8_t* priority,
                     int32_t min_points, int32_t* d_scene_expert, void* cuda_stream);

/* Turns the side stream of emc2_bridge_run off (0) or on (non-zero, the default).  Off, every
 * kernel of the call is enqueued on `cuda_stream` itself, one after another: for callers that
 * want no second stream, and for timing kernels one at a time. */
int emc2_bridge_set_overlap(emc2_bridge_t* bridge, int enable);

/* Stages 3 and 4 for callers that must not allocate device memory (the paper has no counterpart;
 * this is a packaging variant of emc2_route_dispatch).
 *
 * emc2_bridge_create() obtains its scratch with cudaMalloc.  Some hosts cannot do that at the point
 * where they need the dispatch: a plug-in running inside an engine that owns the whole device heap
 * and forbids allocation outside its own pool, or a real-time loop that may not take the driver's
 * allocation lock.  This entry point needs no handle and calls no allocator of any kind: its only
 * scratch (the per-tile expert histograms and their prefix sums) lives in a fixed array that is
 * part of the library image, EMC2_STATIC_SCRATCH_BYTES in size, which every device that loads the
 * library holds from load until the process exits.
 *
 * Arguments and outputs are exactly those of emc2_route_dispatch; in place of the handle it reads,
 * from `config` (HOST memory), only device, point_floats, feat_c, num_thresholds, thresholds,
 * num_experts and lut (other fields are ignored).  All buffers are the caller's.
 *   - Size limit: B * ceil(N / 256) * num_experts must not exceed EMC2_STATIC_SCRATCH_ENTRIES;
 *     a larger call returns EMC2_ERR_TOO_LARGE and enqueues nothing (B <= EMC2_MAX_BATCH still
 *     applies; there is no max_points).
 *   - The first call on each device looks up the array's device address (one runtime query, no
 *     allocation); make that first call outside any stream capture.
 *   - The array is shared by every call in the process and keeps whatever the previous call left;
 *     each call overwrites all entries it later reads, so nothing has to be cleared.  Two calls
 *     whose kernels can overlap on the same device (different streams) race on it: order them.
 * Errors: EMC2_ERR_INVALID_ARG, EMC2_ERR_BAD_CONFIG (of the fields listed), EMC2_ERR_TOO_LARGE,
 * EMC2_ERR_CUDA. */
#define EMC2_STATIC_SCRATCH_ENTRIES (1 << 18)
#define EMC2_STATIC_SCRATCH_BYTES (2 * EMC2_STATIC_SCRATCH_ENTRIES * 4)
int emc2_route_dispatch_static(const emc2_config_t* config, int32_t B, int32_t N, const float* d_points,
                               const uint8_t* d_vis_mask, const float* d_gathered, uint8_t* d_expert,
                               int32_t* d_offsets, int32_t* d_perm, float* d_points_out,
                               float* d_feat_out, void* cuda_stream);

/* Waits for `cuda_stream`, then returns and clears the sticky device status: EMC2_OK,
 * EMC2_ERR_CAPACITY, EMC2_ERR_TIMEOUT or EMC2_ERR_CUDA. */
int emc2_bridge_status(emc2_bridge_t* bridge, void* cuda_stream);

/* Frees scratch memory.  The caller must have synchronised the streams it used.  NULL is OK. */
int emc2_bridge_destroy(emc2_bridge_t* bridge);

/* Text for a status code (static storage, never NULL). */
const char* emc2_status_string(int status);

/* cudaError_t of the last failed runtime call on this handle (0 if none). */
int emc2_bridge_last_cuda_error(const emc2_bridge_t* bridge);

/* Bytes of device scratch the handle owns. */
size_t emc2_bridge_scratch_bytes(const emc2_bridge_t* bridge);

/* Measurement aids (no paper counterpart).  The library counts its own kernel launches per
 * kernel kind; with profiling enabled every launch is also bracketed by CUDA events on the
 * launching stream.  emc2_bridge_profile_read() synchronises those events and fills, for
 * kernel kind k in [0, emc2_bridge_kernel_kinds()), the launches and the summed device
 * milliseconds since the last reset (ms only while profiling was enabled); it then resets
 * the counters if `reset` is non-zero.  Arrays are HOST memory and may be NULL. */
int emc2_bridge_kernel_kinds(void);
const char* emc2_bridge_kernel_name(int kind);
int emc2_bridge_profile_enable(emc2_bridge_t* bridge, int enable);
int emc2_bridge_profile_read(emc2_bridge_t* bridge, int64_t* launches, double* ms, int reset);

/* With profiling enabled: the launches recorded since the last profile_read / profile_timeline, in
 * the order they were enqueued, each with the device time at which it began and ended, in
 * milliseconds after the first of them began (events on the launching streams, so launches on
 * the side stream of emc2_bridge_run show where they ran beside the others).  Fills at most
 * `capacity` entries of the HOST arrays kinds / start_ms / end_ms, returns the number filled (or a
 * negative status) and consumes the records like emc2_bridge_profile_read. */
int emc2_bridge_profile_timeline(emc2_bridge_t* bridge, int32_t* kinds, float* start_ms, float* end_ms,
                                 int32_t capacity);

/* Choice between implementations that produce the same outputs (measurement aid, no paper
 * counterpart; the defaults are the measured winners).  Returns EMC2_ERR_INVALID_ARG for an unknown
 * knob or a value outside its range. */
typedef enum {
    EMC2_TUNE_ROW_STORE = 0,    /* how the one-call path stores feature rows: 0 = 128-bit stores from
                                   registers; 1 = rows staged in shared memory, ordered by expert, and written
                                   with bulk asynchronous copies (cp.async.bulk), both destinations; 2 = bulk
                                   copies for the dispatched rows only; 3 = 256-bit loads and stores
                                   (eight channels per thread; needs feat_c % 8 == 0 and 32-byte aligned
                                   buffers, else falls back to 0) */
    EMC2_TUNE_MARK_IN_PROJECTION = 1, /* emc2_bridge_run: 1 (default) = the projection kernel also marks the
                                   voxel cells of both scales (one pass over the points fewer in stage 1);
                                   0 = stage 1 marks them in a pass of its own, beside the projection */
    EMC2_TUNE_DEDUP_FINE = 2,    /* how the voxels of grid[0] are deduplicated and ranked: 0 (default) = a
                                   direct-addressed cell store (one bit per cell) ranked by prefix sums;
                                   1 = an open-addressing hash table in device memory, sized by the points,
                                   whose unique cell ids are then radix-sorted into canonical order;
                                   2 = a radix sort of every point's (cell id, index).  Same outputs.
                                   Selecting 1 or 2 allocates that design's scratch (this call may allocate;
                                   emc2_bridge_scratch_bytes then includes it) */
    EMC2_TUNE_DEDUP_PILLARS = 3, /* the same choice for grid[1] (default 0 = a direct per-cell count table) */
    EMC2_TUNE_SPLIT_BATCH = 4,   /* emc2_bridge_run with the side stream and B >= 2: 1 = the batch is
                                   projected in two halves, the second on the side stream beside the row
                                   pass of the first; 0 (default) = all frames are projected before any row
                                   moves */
    EMC2_TUNE_KNOBS
} emc2_tuning_t;
int emc2_bridge_set_tuning(emc2_bridge_t* bridge, int32_t knob, int32_t value);

#ifdef __cplusplus
}
#endif
#endif /* EMC2_BRIDGE_H */
