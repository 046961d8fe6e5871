// Device-side data layout shared by the pack, camera and render kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace mv {

// Face codes: 0..5 = -x,+x,-y,+y,-z,+z (outward normal), 6 = camera inside the solid.
constexpr int kFaces = 7;
constexpr int kFaceInside = 6;

constexpr uint32_t kFlagMaterial = 0x1u;
constexpr uint32_t kFlagBoxCount = 0x2u;
constexpr uint32_t kFlagBadCamera = 0x4u;
constexpr uint32_t kFlagTimeout = 0x8u;

// Per-observation ray basis written by the camera kernel (64 bytes, one 128-bit lane each).
struct __align__(16) CamRec {
    float P[3], F[3], Rs[3], Us[3];   // eye, unit forward, per-half-pixel right and up steps
    int32_t self_box;
    uint32_t flags;                   // kFlagBadCamera when a component was not finite
    uint32_t pad[2];
};
static_assert(sizeof(CamRec) == 64, "CamRec must be 64 bytes");

// One environment's render inputs, contiguous in HBM so that a single bulk copy stages them
// into shared memory:  [occupancy bits | shade LUT | boxes | box count + occupied bounds].
// Occupancy is packed along y: the (x, z) column owns 2^ysh consecutive bits (2^ysh >= grid_y, at
// least 32), bit index u = ((x + grid_x*z) << ysh) | y, bit u&31 of word u>>5.  A walk along x or z
// therefore moves by whole words and a walk along y stays inside the column's word(s); for grids
// up to 32 voxels high a column is exactly one word.  The material store uses the same index u.
struct EnvLayout {
    uint32_t occ_bytes;     // grid_x*grid_z*2^ysh/8
    uint32_t lut_off;       // 7*palette_size RGBX words
    uint32_t box_off;       // max_boxes * 32 bytes
    uint32_t count_off;     // 32 bytes: {box count, lo x,y,z, hi x,y,z, pad}; [lo, hi) = cell box
                            // that contains every filled voxel (lo > hi when the grid is empty)
    uint32_t block_bytes;   // bytes staged per CTA (multiple of 16)
    uint32_t stride;        // distance between envs in HBM (multiple of 128)
    uint32_t ysh;           // log2 of the bits per (x, z) column
};

__host__ __device__ __forceinline__ uint32_t voxel_index(uint32_t ysh, int gx, int x, int y, int z) {
    return ((uint32_t)(x + gx * z) << ysh) | (uint32_t)y;
}

struct RenderParams {
    const unsigned char *env_blocks;   // [E] EnvLayout blocks
    const uint8_t *mat;                // [E][grid_x*grid_z << ysh] material ids by voxel index (clamped at upload)
    const CamRec *cams;                // [O]
    uint8_t *rgb;                      // [O][H][W][3]
    float *depth;                      // [O][H][W]
    uint32_t *status;
    EnvLayout lay;
    int obs_begin, obs_count;
    int agents;
    int gx, gy, gz;
    int max_boxes, palette;
    int W, H, tiles_x, tiles_y, mask_words;
    uint32_t sky_rgbx;
    float miss_depth;
    int agents_per_cta;                // observations one CTA renders: 1, or all agents of its env
    int max_steps;                     // most steps a walk can take: grid_x + grid_y + grid_z + 3 (sizes the exit margin)
    float exit_scale;                  // 1 - (bound on the rounding drift of accumulated crossing times)
    // shared-memory offsets after the staged env block: tile table, per-agent blocks (camera record,
    // DDA start table, eye-relative boxes, then overlay rectangles, per-tile box masks and per-tile
    // overlay bits at the offsets below), barrier and flag words
    uint32_t smem_tile_off, smem_agent_off, smem_misc_off;
    uint32_t agent_stride, agent_ov_off, agent_mask_off, agent_ovtile_off;
    const int4 *overlay;               // [O][max_overlay] 16-byte records, or null
    const int32_t *overlay_count;      // [O]
    int max_overlay;
    int wait_polls;                    // bound of the staging wait
    int skip_staging;                  // test hook: the block copy is not issued, so the wait runs out
};

}  // namespace mv
