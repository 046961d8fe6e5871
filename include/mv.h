/*
 * mv.h — C ABI of the B200 batched RGB-D renderer for voxel-grid worlds.
 *
 * The library implements the Render half of the paper's batched simulation step
 * (Section 3.2, Eq. 2: O(t+1) = Render(S(t+1))) for N environments x M agents in one call
 * (Section 3.2; Appendix A.1: one step returns N x M observations).  The state of one
 * environment is the discretised world of Section 3.1 (a voxel grid) plus the movable
 * entities of Section 3.2 (interactive objects and agent bodies) as axis-aligned boxes, plus
 * one camera per agent.  Observations are W x H RGB frames (Appendix A.2: 128 x 72 x 3) with
 * an added float depth channel.  The paper renders with a batched rasteriser; this library
 * casts one primary ray per pixel centre, which yields the same visible surface.
 *
 * Geometry conventions (the paper leaves them open):
 *   - y is up.  Voxel (i,j,k) is the unit cube [i,i+1] x [j,j+1] x [k,k+1]; the grid starts
 *     at the world origin.  Input grids are uint8 material ids, 0 = empty, laid out
 *     [env][j (y)][k (z)][i (x)] with x fastest.
 *   - yaw 0 looks along +z and grows toward +x; pitch > 0 looks up; image row 0 is the top.
 *   - depth is planar: distance along the view axis, in voxel units.  A pixel that hits
 *     nothing gets sky_rgb and miss_depth.  A camera inside a solid gets depth 0 and the
 *     ambient-only colour of that solid.
 *   - colour = palette[env][material] * (ambient + (1-ambient) * max(0, n . L)), L the unit
 *     direction to the light, n the face normal, rounded half up to uint8 (evaluated in
 *     double when palettes are uploaded).
 *   - observation index = env * agents_per_env + agent.
 *
 * Memory and ownership.  Every pointer named d_* is DEVICE memory owned by the caller; the
 * library reads or writes it only inside the stream work the call enqueues and never keeps
 * it.  Every pointer named h_* is HOST memory owned by the caller.  Output buffers must be
 * 16-byte aligned.  The library owns only what mv_create_batch allocates; mv_destroy frees it.
 *
 * Asynchrony.  All device work is enqueued on the cuda_stream argument (a cudaStream_t cast to
 * void*, NULL = the legacy default stream).  Calls do not synchronise, except mv_query_status,
 * mv_step_host and mv_destroy.
 *
 * Errors.  Every call returns MV_OK (0) or a negative mv_status.  Nothing throws or aborts.
 * Bad data (material id >= palette_size, box count > max_boxes, non-finite camera) never causes
 * an out-of-bounds access: ids and counts are clamped, a non-finite camera renders a sky frame,
 * and a sticky bit is set in the device status word (see mv_query_status).
 */
#ifndef MV_H
#define MV_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum mv_status {
    MV_OK = 0,
    MV_ERR_INVALID_ARG = -1,     /* null pointer, size out of range, bad descriptor */
    MV_ERR_OUT_OF_MEMORY = -2,   /* device or host allocation failed */
    MV_ERR_CUDA = -3,            /* a CUDA runtime call failed */
    MV_ERR_NOT_READY = -4,       /* render before every env has a grid and palette, or before cameras */
    MV_ERR_DEVICE_TIMEOUT = -5,  /* a bounded device-side wait gave up (reported by mv_query_status) */
    MV_ERR_UNSUPPORTED = -6      /* configuration exceeds a documented limit */
} mv_status;

/* Sticky data-error bits returned (as a positive value) by mv_query_status. */
#define MV_FLAG_MATERIAL_CLAMPED 0x1u   /* a voxel or box material id was >= palette_size */
#define MV_FLAG_BOX_COUNT_CLAMPED 0x2u  /* a box count was > max_boxes or negative */
#define MV_FLAG_BAD_CAMERA 0x4u         /* a camera had a non-finite component */
#define MV_FLAG_DEVICE_TIMEOUT 0x8u     /* a staging wait in the render kernel timed out */

typedef struct mv_batch mv_batch;       /* opaque; owned by the library */

/* A movable entity of Section 3.2 reduced to an axis-aligned box.  32 bytes.
 * A box with min >= max on any axis is ignored. */
typedef struct mv_box {
    float min[3];
    float max[3];
    uint32_t material;                  /* palette index */
    uint32_t pad;
} mv_box;

/* One agent camera.  24 bytes.  self_box is the index (within the env's box list) of the
 * agent's own body, which this camera does not see; -1 for none. */
typedef struct mv_camera {
    float pos[3];
    float yaw, pitch;                   /* radians */
    int32_t self_box;
} mv_camera;

/* One filled rectangle of the pixel-space GUI (paper Appendix A.2: bars and indicators drawn in
 * the agent's field of view, e.g. the time-left bar).  Pixel coordinates, half-open
 * [x0,x1) x [y0,y1), clipped to the image.  16 bytes. */
typedef struct mv_overlay_rect {
    int16_t x0, y0, x1, y1;
    uint8_t rgb[3];
    uint8_t pad0;
    uint32_t pad1;
} mv_overlay_rect;

/* One agent's motion command for a step (paper Appendix A.2, action table: moving, strafing,
 * turning, vertical gaze), already scaled to world units and radians.  16 bytes. */
typedef struct mv_agent_move {
    float forward, strafe;              /* along the horizontal view direction / to the right */
    float dyaw, dpitch;
} mv_agent_move;

/* Agent body used for collision: the box [x-half_width, x+half_width] x
 * [y-below_eye, y+above_eye] x [z-half_width, z+half_width] around the eye. */
typedef struct mv_body_shape {
    float half_width, below_eye, above_eye;
    float max_pitch;                    /* |pitch| is clamped to this */
} mv_body_shape;

typedef struct mv_batch_desc {
    int32_t num_envs;                   /* N >= 1 */
    int32_t agents_per_env;             /* M >= 1 */
    int32_t grid_x, grid_y, grid_z;     /* voxels per axis; each a multiple of 4, 4..1024.
                                           The occupancy bits are kept packed along y, one
                                           column of h bits per (x, z), h = the power of two
                                           >= grid_y, at least 32.  While grid_x*grid_z*h/8 bytes
                                           plus the per-env tables fit in shared memory (about
                                           200 KB) they are staged there; larger grids are read
                                           from global memory (slower per step, same results).
                                           Grids up to 32 high take the fastest traversal. */
    int32_t max_boxes;                  /* per env, agent bodies included; 0..256 */
    int32_t width, height;              /* pixels; width a multiple of 8, height of 4; <= 4096 */
    int32_t palette_size;               /* 1..256 entries per env */
    float hfov_rad;                     /* horizontal field of view, (0, pi) */
    float light_dir[3];                 /* direction TO the light; any non-zero length */
    float ambient;                      /* [0, 1] */
    uint8_t sky_rgb[3];
    uint8_t pad;
    float miss_depth;
    int32_t device;                     /* CUDA device ordinal */
    int32_t max_overlay_rects;          /* GUI rectangles per observation, 0..16 (0 = no overlay) */
} mv_batch_desc;

/* Allocate the device-resident world store, camera table and status word for a batch
 * (paper Section 3.2: one instance hosts N environments with M agents each).
 * desc: HOST pointer.  out: HOST pointer receiving the handle.
 * Errors: INVALID_ARG (null, out-of-range field), UNSUPPORTED (tile masks, boxes and tables of one
 * observation exceed shared memory, e.g. a very large image), OUT_OF_MEMORY, CUDA. */
int mv_create_batch(const mv_batch_desc *desc, mv_batch **out);

/* Upload world state for envs [env_begin, env_begin+env_count) (paper Section 3.3: geometry
 * is prepared once per episode; Section 3.1: objects move every step, hence any of the array
 * arguments may be NULL meaning "keep what was uploaded before").
 *   d_grid      DEVICE uint8 [env_count][grid_y][grid_z][grid_x]; packed on the device into a
 *               1-bit occupancy grid plus a material store.
 *   d_boxes     DEVICE mv_box [env_count][max_boxes]
 *   d_box_count DEVICE int32 [env_count]; required when d_boxes is given
 *   d_palette   DEVICE uint8 [env_count][palette_size][3]; the per-env shaded colour table
 *               is rebuilt from it on the device
 * Errors: INVALID_ARG (range, d_boxes without d_box_count), CUDA. */
int mv_upload_worlds(mv_batch *batch, int env_begin, int env_count, const uint8_t *d_grid,
                     const mv_box *d_boxes, const int32_t *d_box_count, const uint8_t *d_palette,
                     void *cuda_stream);

/* The same upload for envs that are not neighbours (paper Appendix A.1: environments end their
 * episodes at different steps and are reset on their own): env i of the arrays goes to env
 * h_env_index[i] of the batch.
 *   h_env_index HOST int32 [env_count], strictly increasing, each in [0, num_envs).  It is copied to
 *               the device in stream order; if it lies in pinned memory the caller keeps it unchanged
 *               until the stream has passed this call.  The batch owns one device buffer for it, so
 *               scattered uploads of one batch go to one stream at a time.
 *   the other arguments: as for mv_upload_worlds, indexed by i.
 * No counterpart in the paper's interface (its environments reset inside the simulator).
 * Errors: INVALID_ARG (null list, index out of range or not increasing, d_boxes without
 * d_box_count), CUDA. */
int mv_upload_worlds_at(mv_batch *batch, int env_count, const int32_t *h_env_index, const uint8_t *d_grid,
                        const mv_box *d_boxes, const int32_t *d_box_count, const uint8_t *d_palette,
                        void *cuda_stream);

/* Set all cameras (paper Section 3.2: cameras are part of the state; Appendix A.1: N x M
 * observations per step) and build each one's ray basis on the device.
 *   d_cams DEVICE mv_camera [num_envs*agents_per_env]
 * Errors: INVALID_ARG, CUDA. */
int mv_set_cameras(mv_batch *batch, const mv_camera *d_cams, void *cuda_stream);

/* Render every observation of the batch in one launch (paper Section 3.2, Eq. 2; "a single
 * request to the GPU to render all the observations").
 *   d_rgb   DEVICE uint8 [num_obs][height][width][3]
 *   d_depth DEVICE float [num_obs][height][width]
 * Errors: INVALID_ARG, NOT_READY (some env has no grid/palette yet, or no cameras), CUDA. */
int mv_render_batch(mv_batch *batch, uint8_t *d_rgb, float *d_depth, void *cuda_stream);

/* Merge the voxels of envs [env_begin, env_begin+env_count) into boxes (paper Section 3.3: at
 * the start of an episode adjacent voxels are merged greedily into a small number of enclosing
 * parallelepipeds).  The render path of this library walks the grid and does not need the
 * merged form; the boxes are for callers that want the paper's compact geometry (a rasteriser, a
 * physics broad phase) or want to compare box primitives with grid traversal.  Order and shape are
 * those of a serial sweep in index order (x fastest, then z, then y) that grows each box along
 * +x, then +z, then +y over cells of one material.
 *   d_boxes_out DEVICE mv_box [env_count][max_out]; box b of an env is valid for b < min(count, max_out)
 *   d_count_out DEVICE int32 [env_count]; the number of boxes the sweep produces (may exceed max_out,
 *               in which case only the first max_out were written)
 * The first call allocates scratch (2 bits per voxel for as many envs as fit in 1 GiB, at most the batch: the
 * coverage bitmap and a copy of the occupancy in sweep order).
 * Errors: INVALID_ARG, NOT_READY (an env in the range has no grid), OUT_OF_MEMORY, CUDA. */
int mv_merge_voxels(mv_batch *batch, int env_begin, int env_count, mv_box *d_boxes_out,
                    int32_t *d_count_out, int max_out, void *cuda_stream);

/* Set the GUI overlay of every observation (paper Appendix A.2).  The rectangles are painted
 * over the RGB frame in list order (later ones on top) by the render kernel's store stage; depth
 * is not touched.  The overlay stays in force until set again.
 *   d_rects DEVICE mv_overlay_rect [num_obs][max_overlay_rects], or NULL to clear all overlays
 *   d_count DEVICE int32 [num_obs] rectangles in use per observation (clamped to
 *           0..max_overlay_rects); required when d_rects is given
 * Errors: INVALID_ARG (d_rects without d_count, or the batch was created with
 * max_overlay_rects == 0 and d_rects is not NULL), CUDA. */
int mv_set_overlays(mv_batch *batch, const mv_overlay_rect *d_rects, const int32_t *d_count,
                    void *cuda_stream);

/* Move every agent and collide its body with the voxel grid (paper Section 3.1: agent movement
 * and collision checking are continuous; Section 3.2, Eq. 1, the agent part of
 * S' = Physics(S, A)), then rebuild its ray basis, so that mv_render_batch can follow directly.
 * Per agent: yaw += dyaw; pitch = clamp(pitch + dpitch); the horizontal step
 * forward*(sin yaw, cos yaw) + strafe*(cos yaw, -sin yaw) is evaluated in double and added to the
 * float position; the x move is kept iff the body at the new x lies inside the grid and touches
 * no filled voxel, then the z move likewise from the accepted x (axis-separated sliding).  Movable
 * boxes do not block.  If the camera's self_box is a valid box index, that box is moved with the
 * body (material kept) so that other agents see it.
 *   d_cams_inout DEVICE mv_camera [num_obs], updated in place (the caller owns agent state)
 *   d_moves      DEVICE mv_agent_move [num_obs]
 *   shape        HOST pointer, or NULL for {0.25, 0.75, 0.25, max_pitch 1.0}
 * Needs the grids of all envs (NOT_READY otherwise).  Errors: INVALID_ARG, NOT_READY, CUDA. */
int mv_move_agents(mv_batch *batch, mv_camera *d_cams_inout, const mv_agent_move *d_moves,
                   const mv_body_shape *shape, void *cuda_stream);

/* One whole step from HOST memory (paper Section 3.2: by default the rendered frames are
 * transferred to CPU memory): copies cameras (and, if given, this step's boxes) host->device,
 * builds ray bases, renders, and copies rgb and depth device->host, overlapping the copies with
 * rendering chunk by chunk.  Synchronous: on return the host buffers hold the frames.
 *   h_cams      HOST mv_camera [num_obs]
 *   h_boxes     HOST mv_box [num_envs][max_boxes] or NULL (keep)
 *   h_box_count HOST int32 [num_envs]; required when h_boxes is given
 *   h_rgb, h_depth HOST outputs, same shapes as mv_render_batch; page-locked memory is
 *               needed for the copies to overlap
 * The first call allocates device-side frame buffers of the batch's full output size (all of
 * them or, on failure, none: a failed first call can be retried).
 * Errors: as the calls it is made of; DEVICE_TIMEOUT if a bounded device-side wait ran out during
 * the step (the frames are then not valid; the flag stays set until mv_query_status clears it). */
int mv_step_host(mv_batch *batch, const mv_camera *h_cams, const mv_box *h_boxes,
                 const int32_t *h_box_count, uint8_t *h_rgb, float *h_depth, void *cuda_stream);

/* One whole step from HOST memory for callers that must not allocate.  (The paper has no
 * counterpart; this exists for deployment.)  Some hosts of this library cannot call cudaMalloc
 * once they are running: a trainer that has handed every free byte of the GPU to its own memory
 * pool, a control loop that cannot afford the device-wide synchronisation an allocation may
 * cause, or a process whose policy forbids allocation after start-up.  mv_step_host allocates
 * frame buffers on its first call; this variant never allocates.  It stages the cameras and the
 * rendered frames in a fixed 8 MiB array that is part of the library image (so every GPU that
 * loads the library carries those 8 MiB until the process exits) and otherwise does what
 * mv_step_host does without the box update: cameras in, ray bases, render, frames out.
 *   h_cams  HOST mv_camera [num_obs]
 *   h_rgb, h_depth HOST outputs, shapes as in mv_render_batch
 * Limit: num_obs * (7*width*height + 24) bytes, with the two frame buffers each rounded up to
 * 256 bytes, must fit in 8 MiB (129 observations at 128x72); a larger batch gets
 * MV_ERR_UNSUPPORTED and nothing runs.  The batch must have been created and its worlds
 * uploaded beforehand, when allocating was still allowed.
 * The first call on each device looks up the array's device address (a runtime query, not an
 * allocation); make that first call before starting any stream capture.
 * The array is shared by every batch and every call on that device and keeps whatever the last
 * call left in it.  Nothing in it needs clearing, because each call that returns MV_OK has
 * overwritten every byte it read back; but two calls whose device work overlaps (different streams, or different
 * threads) race on it, so serialise them.  Synchronous like mv_step_host.
 * Calls no cudaMalloc, cudaFree or other allocating routine.
 * Errors: INVALID_ARG, NOT_READY, UNSUPPORTED (batch too large for the array, device ordinal
 * >= 64), DEVICE_TIMEOUT (as mv_step_host; the array may then hold an earlier call's frames),
 * CUDA. */
int mv_step_host_static(mv_batch *batch, const mv_camera *h_cams, uint8_t *h_rgb, float *h_depth,
                        void *cuda_stream);

/* Synchronise the stream and return the device status word: a negative mv_status if a CUDA
 * error or device timeout occurred, else the OR of the MV_FLAG_* bits seen so far (0 = clean).
 * clear != 0 resets the sticky bits. */
int mv_query_status(mv_batch *batch, int clear, void *cuda_stream);

/* Number of kernels of this library launched on behalf of `batch` so far (host counter). */
int64_t mv_launch_count(const mv_batch *batch);

/* ---- Test and measurement hooks (no counterpart in the paper).  They are exported by the library but
 * declared only for translation units that define MV_ENABLE_TEST_HOOKS before including this header;
 * they change how the render kernel runs, never what it computes.  Host-only calls. */
#ifdef MV_ENABLE_TEST_HOOKS

/* on != 0 makes the render kernel read the occupancy bits from global memory instead of staging them
 * in shared memory, which is what happens by itself for grids too large for shared memory; on == 0
 * restores staging (UNSUPPORTED if the grid does not fit).  Results are identical either way. */
int mv_debug_occupancy_in_global(mv_batch *batch, int on);

/* Failure-detection hook.  The render kernel's only device-side wait is the bounded wait for the
 * staged env block; with skip_staging != 0 the copy is not issued, so every CTA's wait runs out after
 * wait_polls polls, the kernel returns without touching the outputs and MV_FLAG_DEVICE_TIMEOUT is set
 * (mv_query_status then returns MV_ERR_DEVICE_TIMEOUT).  Nothing faults or hangs and the context stays
 * usable.  Defaults: skip_staging 0, wait_polls 2^18; wait_polls must be in 1..2^24.
 * Errors: INVALID_ARG. */
int mv_debug_staging(mv_batch *batch, int skip_staging, int wait_polls);

/* How many observations one CTA of the render kernel renders: 1 (a CTA per observation) or
 * agents_per_env (a CTA per environment, its block staged once for all its agents); 0 restores the
 * library's own choice, which depends on how many environments the batch has.  Results are identical.
 * Errors: INVALID_ARG (any other value), UNSUPPORTED (the per-environment shape does not fit shared
 * memory). */
int mv_debug_agents_per_cta(mv_batch *batch, int agents_per_cta);

#endif /* MV_ENABLE_TEST_HOOKS */

/* Free everything mv_create_batch allocated (synchronises the device). NULL is accepted. */
int mv_destroy(mv_batch *batch);

/* Static, never-freed description of a status code. */
const char *mv_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* MV_H */
