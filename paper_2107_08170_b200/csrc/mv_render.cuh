// The render kernel: ray generation, grid traversal, box tests, shading and frame store for
// every observation of the batch in one launch (paper Section 3.2, Eq. 2).
//
// One CTA renders the observations of one environment (all of its agents, or one agent when the
// batch has too few environments to fill the GPU that way).  A single bulk asynchronous copy
// stages the environment's block (1-bit occupancy grid, shaded colour table, box list) into
// shared memory once for all of them; while it is in flight the CTA clears the per-tile box
// masks and writes the tile table.  Each agent's boxes are then binned to 8x4-pixel screen tiles
// by the bounding rectangle of their projected corners (conservative, so every box that a
// pixel's ray can touch is tested for that pixel).  Tiles are dealt to warps round-robin; each
// lane owns one pixel of the tile: it walks the occupancy grid (packed along y: a column of up to
// 32 voxels is one word) with a predicated 3D-DDA in shared memory, tests the tile's candidate
// boxes with slab tests, looks the colour up in the shaded table and the warp writes 24-byte RGB
// row segments as packed 32-bit words and 32-byte depth row segments.  The common case runs in
// three blocks of PTX (ray set-up + walk, colour, stores); everything rarer is C++ around them.
// The walk is confined to the cell box that holds every filled voxel of the environment (built at
// upload), so rays that leave it stop at once; GUI rectangles, if any, are painted over the colour
// just before the store.
#pragma once
#include "mv_device.cuh"

namespace mv {

__device__ __forceinline__ uint32_t smem_addr(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
// Plain (single-CTA) bulk copy global -> shared, completion counted on an mbarrier.
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after `limit` polls instead of spinning forever.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity, int limit) {
    for (int i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

#define kInf (__int_as_float(0x7f800000))
constexpr uint32_t kNoRow = 0xffffffffu;           // "no surface" marker of the traversal
constexpr int kDrainPolls = 1 << 26;               // bound of the wait for a copy known to be in flight

// Reciprocal to 1 ulp in one instruction; every use is inside toleranced intersection arithmetic.
__device__ __forceinline__ float fast_rcp(float x) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
// Makes a value opaque to the optimiser at this point, so that it is held in a register from
// here on instead of being recomputed at every use.
template <typename T> __device__ __forceinline__ void keep(T &v) { asm volatile("" : "+r"(reinterpret_cast<uint32_t &>(v))); }
template <typename T> __device__ __forceinline__ void keep64(T *&v) { asm volatile("" : "+l"(v)); }
__device__ __forceinline__ float min3f(float a, float b, float c) {
    float r;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
__device__ __forceinline__ float max3f(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// ---------------------------------------------------------------------------------------------
// The DDA loop.  Crossing times accumulate (t += dt) and the exit time handed in is pulled in by
// the rounding drift that can build up, which keeps the walk inside the occupied box; the loop is
// also bounded by a step budget.  One step: t = min(tx,ty,tz); leave when t >= exit time or when
// the cell entered by the previous step is filled (one branch for both); else the axis whose
// crossing time equals t (ties: x, then y, then z) advances.  Two registers alternate as t, so
// that after a hit the time at which the filled cell was entered is still there.
//
// Two flavours of the cell state:
//  * column-word (grids up to 32 voxels high, occupancy in shared memory): the state is the
//    shared-memory address `pos` of the (x, z) column's word and a one-bit mask `bit` of the height;
//    x and z steps add a byte stride to the address, a y step rotates the mask by 1 or 31, and the
//    test is one load and one AND.
//  * indexed (any grid): the state is the voxel index `pos` (plus 8x the shared-memory byte address
//    of the occupancy when it is staged, so that (pos >> 3) & ~3 is the word's address and pos & 31
//    the bit); every step adds a stride.
// Register names used by the macros (declared by the enclosing asm block): tx ty tz dtx dty dtz
// (f32), sx sy sz pos bit w a it (b32), ta tb (f32), px py pz pq ph pf (pred), texit (f32); the
// global flavour also uses ag (b64) and the operand named by MV_DDA_GBASE.
#if defined(MV_PROBE) && MV_PROBE == 9
#define MV_DDA_COUNT " add.f32 ns, ns, 0f3F800000;\n"
#else
#define MV_DDA_COUNT
#endif
#if defined(MV_TEST_FORM) && MV_TEST_FORM == 1
#define MV_DDA_TESTBIT " and.b32 w, w, bit;\n setp.ne.u32 ph, w, 0;\n"
#else
#define MV_DDA_TESTBIT " lop3.or.b32 w|ph, w, bit, 0, 0xC0, pf;\n"
#endif
#define MV_DDA_HEAD(T, OUT)                          \
    " min.f32 " T ", tx, ty, tz;\n"                  \
    " setp.geu.or.f32 pq, " T ", texit, ph;\n"       \
    " @pq bra " OUT ";\n"                            \
    MV_DDA_COUNT                                     \
    " setp.eq.f32 px, tx, " T ";\n"                  \
    " setp.eq.and.f32 py|pz, ty, " T ", !px;\n"      \
    " @px add.f32 tx, tx, dtx;\n"                    \
    " @py add.f32 ty, ty, dty;\n"                    \
    " @pz add.f32 tz, tz, dtz;\n"
#define MV_DDA_STEP_COLW(T, OUT) MV_DDA_HEAD(T, OUT)  \
    " @px add.s32 pos, pos, sx;\n"                   \
    " @pz add.s32 pos, pos, sz;\n"                   \
    " @py shf.l.wrap.b32 bit, bit, bit, sy;\n"       \
    " ld.shared.u32 w, [pos];\n"                     \
    MV_DDA_TESTBIT
#define MV_DDA_STEP_IDX_TAIL                         \
    " shf.r.wrap.b32 w, w, 0, pos;\n"                \
    " lop3.or.b32 w|ph, w, 1, 0, 0xC0, pf;\n"
#define MV_DDA_STEP_IDX_ADV                          \
    " @px add.s32 pos, pos, sx;\n"                   \
    " @py add.s32 pos, pos, sy;\n"                   \
    " @pz add.s32 pos, pos, sz;\n"
#define MV_DDA_STEP_IDX(T, OUT) MV_DDA_HEAD(T, OUT) MV_DDA_STEP_IDX_ADV \
    " shr.u32 a, pos, 3;\n and.b32 a, a, 0xfffffffc;\n ld.shared.u32 w, [a];\n" MV_DDA_STEP_IDX_TAIL
#define MV_DDA_STEP_IDX_GLOBAL(T, OUT) MV_DDA_HEAD(T, OUT) MV_DDA_STEP_IDX_ADV \
    " shr.u32 a, pos, 5;\n mad.wide.u32 ag, a, 4, gbase;\n ld.global.nc.u32 w, [ag];\n" MV_DDA_STEP_IDX_TAIL
// Loop around eight steps.  On leaving: ph = a filled cell was entered, thit = when, and px/py
// still say along which axis.
#define MV_DDA_LOOP(STEP)                            \
    " setp.ne.u32 pf, 0, 0;\n"                       \
    " setp.ne.u32 ph, 0, 0;\n"                       \
    "MV_DDA_LOOP_TOP:\n"                             \
    STEP("ta", "MV_DDA_OUT_A") STEP("tb", "MV_DDA_OUT_B") STEP("ta", "MV_DDA_OUT_A") STEP("tb", "MV_DDA_OUT_B") \
    STEP("ta", "MV_DDA_OUT_A") STEP("tb", "MV_DDA_OUT_B") STEP("ta", "MV_DDA_OUT_A") STEP("tb", "MV_DDA_OUT_B") \
    " sub.s32 it, it, 8;\n"                          \
    " setp.gt.s32 pq, it, 0;\n"                      \
    " @pq bra MV_DDA_LOOP_TOP;\n"                    \
    "MV_DDA_OUT_A:\n"                                \
    " @ph mov.f32 thit, tb;\n"                       \
    " bra MV_DDA_OUT;\n"                             \
    "MV_DDA_OUT_B:\n"                                \
    " @ph mov.f32 thit, ta;\n"                       \
    "MV_DDA_OUT:\n"
#define MV_DDA_DECL                                  \
    " .reg .pred px, py, pz, pq, ph, pf;\n"          \
    " .reg .f32 tx, ty, tz, dtx, dty, dtz, ta, tb, texit, thit, ns;\n" \
    " .reg .b32 sx, sy, sz, pos, bit, w, a, it;\n"   \
    " .reg .b64 ag, gbase;\n"                        \
    " mov.f32 ns, 0f00000000;\n"

// MV_PROBE builds are for instruction counting only (never the shipped library): 1 = every walk ends
// at its first test, 2 = also no box tests, 3 = no tiles at all (CTA prologue alone), 9 = the depth
// channel carries each ray's number of walk steps instead of depth.
#ifndef MV_PROBE
#define MV_PROBE 0
#endif
// MV_BRICKS builds are an experiment, never the shipped library: 1 = two-level traversal (a one-bit map
// of 4x4x4 bricks built per CTA; empty bricks are jumped across, occupied ones walked cell by cell by
// the same PTX loop), 2 = the flat walk through the same C++ path, as the like-for-like baseline of 1.
// Both need grid_x to be a power of two and a grid at most 32 high.
#ifndef MV_BRICKS
#define MV_BRICKS 0
#endif
#ifndef MV_MINB
#define MV_MINB 3
#endif

constexpr uint32_t kOverlayTileBit = 0x80000000u;   // in a tile's box mask word (only when max_boxes < 32)
constexpr uint32_t kAgentInside = 1u;      // eye inside the occupied cell box
constexpr uint32_t kAgentBad = 2u;         // non-finite camera: sky frame
constexpr uint32_t kAgentFilled = 4u;      // the eye's own voxel is filled
// Per-agent block in shared memory (16-byte slots): camera record (3), {hit time a ray starts with,
// flags, self box, overlay count} (1), {start bit mask, exit-time factor, start colour row, start position} (1), {64-bit address
// of the env's material store, biased for the walk's positions} (1), DDA start
// table (8 sign combinations x 3 axes), then eye-relative boxes, overlay rectangles, per-tile box
// masks and per-tile overlay bits at offsets the host lays out.
constexpr int kAgentRecVecs = 6;
constexpr int kDdaVecs = 24;
// byte offsets, from the agent block's start plus 48 x (sign combination), of the DDA table rows of
// the x, y and z axis and of the colour-row word of the x row (as text, for the PTX blocks)
// hard bound of the traversal loop: no grid allows more steps than 3 x 1024 + 3
#define MV_STEP_BUDGET "3080"
#define MV_TAB_X "96"
#define MV_TAB_Y "112"
#define MV_TAB_Z "128"
#define MV_TAB_ROW "108"
static_assert(16 * kAgentRecVecs == 96, "MV_TAB_* follow the agent record size");
constexpr uint32_t kAgentDdaOff = 16u * kAgentRecVecs;
constexpr uint32_t kAgentRelOff = 16u * (kAgentRecVecs + kDdaVecs);

// One thread's share of a sky frame (non-finite camera).
template <int NT>
__device__ __forceinline__ void write_sky(uint8_t *rgb_obs, float *depth_obs, int npx, uint32_t sky_rgbx, float miss_depth) {
    for (int i = threadIdx.x; i < npx; i += NT) depth_obs[i] = miss_depth;
    for (int i = threadIdx.x; i < npx * 3; i += NT) rgb_obs[i] = (uint8_t)(sky_rgbx >> (8 * (i % 3)));
}

// OCC_SHARED: the occupancy bits are staged in shared memory with the rest of the env block (the
// normal case); otherwise only the block's tail (colour table, boxes, bounds) is staged and the
// occupancy is read from global memory through the read-only path.
// COLW: column-word flavour of the walk (grid at most 32 high and occupancy staged).
template <int NT, bool OCC_SHARED, bool COLW>
__global__ void __launch_bounds__(NT, (MV_MINB * 384) / NT) render_kernel(const RenderParams p)
{
    static_assert(OCC_SHARED || !COLW, "the column-word walk reads shared memory");
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int apc = p.agents_per_cta;
    const int obs0 = p.obs_begin + blockIdx.x * apc;
    const int env = p.agents == 1 ? obs0 : obs0 / p.agents;
    const int W = p.W, H = p.H;
    const int ntiles = p.tiles_x * p.tiles_y;
    // Box masks per tile: mw words of one bit per box.  With more than 32 boxes a summary word (the OR of
    // the others) comes first, so that the per-tile test reads one word whatever the box count.
    const int mw = p.mask_words;
    const int ms = mw > 1 ? mw + 1 : 1;              // words per tile
    const int m0 = mw > 1 ? 1 : 0;                   // position of the first real mask word

    // bytes of the env block that are NOT staged (the occupancy, when it stays in global memory)
    const uint32_t unstaged = OCC_SHARED ? 0u : p.lay.occ_bytes;
    const unsigned char *env_block = p.env_blocks + (size_t)env * p.lay.stride;
    const uint32_t *s_occ = OCC_SHARED ? reinterpret_cast<const uint32_t *>(smem)
                                       : reinterpret_cast<const uint32_t *>(env_block);
    const unsigned char *s_lut = smem + (p.lay.lut_off - unstaged);
    const float4 *s_box = reinterpret_cast<const float4 *>(smem + (p.lay.box_off - unstaged));
    const int *s_count = reinterpret_cast<const int *>(smem + (p.lay.count_off - unstaged));
    float4 *s_tile = reinterpret_cast<float4 *>(smem + p.smem_tile_off);
    unsigned char *s_agents = smem + p.smem_agent_off;
    uint64_t *s_bar = reinterpret_cast<uint64_t *>(smem + p.smem_misc_off);
    uint32_t *s_flag = reinterpret_cast<uint32_t *>(smem + p.smem_misc_off + 8);
    auto agent_rec = [&](int ag) { return reinterpret_cast<float4 *>(s_agents + (size_t)ag * p.agent_stride); };
    auto agent_dda = [&](int ag) { return agent_rec(ag) + kAgentRecVecs; };
    auto agent_rel = [&](int ag) { return agent_rec(ag) + kAgentRecVecs + kDdaVecs; };
    auto agent_ov = [&](int ag) { return reinterpret_cast<int4 *>(s_agents + (size_t)ag * p.agent_stride + p.agent_ov_off); };
    auto agent_mask = [&](int ag) { return reinterpret_cast<uint32_t *>(s_agents + (size_t)ag * p.agent_stride + p.agent_mask_off); };
    auto agent_ovtile = [&](int ag) { return reinterpret_cast<uint32_t *>(s_agents + (size_t)ag * p.agent_stride + p.agent_ovtile_off); };
    const int ovt_words = (ntiles + 31) / 32;

    // ---- stage the environment block
    if (tid == 0) mbar_init(s_bar, 1);
    __syncthreads();
    if (tid == 0 && !p.skip_staging) {
        mbar_expect_tx(s_bar, p.lay.block_bytes - unstaged);
        bulk_load(smem, env_block + unstaged, p.lay.block_bytes - unstaged, s_bar);
    }
    // ---- meanwhile: tile table, cleared masks, camera records, GUI rectangles
    for (int ag = 0; ag < apc; ++ag) {
        uint32_t *mk = agent_mask(ag);
        for (int i = tid; i < ntiles * ms; i += NT) mk[i] = 0u;
    }
    const float inv_tiles_x = 1.0f / (float)p.tiles_x;
    for (int i = tid; i < ntiles; i += NT) {
        // (i + 0.5) / tiles_x is at least 1 / (2 tiles_x) away from an integer: exact in float for any image
        const int ty = (int)(((float)i + 0.5f) * inv_tiles_x), tx = i - ty * p.tiles_x;
        // a = 2px+1-W and b = H-1-2py of the tile's first pixel (small integers: exact as floats)
        s_tile[i] = make_float4((float)(16 * tx + 1 - W), (float)(H - 1 - 8 * ty), __int_as_float(ty * 4 * W + tx * 8),
                                __int_as_float(i));
    }
    for (int ag = tid; ag < apc; ag += NT) {
        const float4 *cq = reinterpret_cast<const float4 *>(p.cams + obs0 + ag);
        const float4 c3 = __ldg(cq + 3);
        float4 *rec = agent_rec(ag);
        rec[0] = __ldg(cq);
        rec[1] = __ldg(cq + 1);
        rec[2] = __ldg(cq + 2);
        const int ovc = p.overlay ? min(max(__ldg(p.overlay_count + obs0 + ag), 0), p.max_overlay) : 0;
        rec[3] = make_float4(0.0f, __uint_as_float((__float_as_uint(c3.y) & kFlagBadCamera) ? kAgentBad : 0u), c3.x,
                             __int_as_float(ovc));
    }
    if (p.overlay) {
        // GUI rectangles of each observation (unpacked to x0,y0,x1,y1 / colour in two slots) and one
        // bit per tile that any rectangle touches, so untouched tiles pay a single bit test
        for (int i = tid; i < apc * ovt_words; i += NT) agent_ovtile(i / ovt_words)[i % ovt_words] = 0u;
        __syncthreads();
        for (int i = tid; i < apc * p.max_overlay; i += NT) {
            const int ag = i / p.max_overlay, r = i - ag * p.max_overlay;
            const int ovc = min(max(__ldg(p.overlay_count + obs0 + ag), 0), p.max_overlay);
            if (r >= ovc) continue;
            const int4 q = __ldg(p.overlay + (size_t)(obs0 + ag) * p.max_overlay + r);
            const int x0 = (int)(short)(q.x & 0xffff), y0 = (int)(short)(q.x >> 16);
            const int x1 = (int)(short)(q.y & 0xffff), y1 = (int)(short)(q.y >> 16);
            agent_ov(ag)[2 * r] = make_int4(x0, y0, x1, y1);
            agent_ov(ag)[2 * r + 1] = make_int4(q.z & 0xffffff, 0, 0, 0);
            const int cx0 = max(x0, 0), cy0 = max(y0, 0), cx1 = min(x1, W), cy1 = min(y1, H);
            if (cx0 < cx1 && cy0 < cy1)
                for (int ty = cy0 >> 2; ty <= ((cy1 - 1) >> 2); ++ty)
                    for (int tx = cx0 >> 3; tx <= ((cx1 - 1) >> 3); ++tx) {
                        const int t = ty * p.tiles_x + tx;
                        atomicOr(&agent_ovtile(ag)[t >> 5], 1u << (t & 31));
                        // with fewer than 32 boxes the top bit of the tile's box mask is free: it sends
                        // exactly the touched tiles down the slow branch
                        if (p.max_boxes < 32) atomicOr(&agent_mask(ag)[t], kOverlayTileBit);
                    }
        }
    }

    // ---- wait for the block: one warp polls, the whole CTA takes the same decision
    if (warp == 0) {
        const bool ok = mbar_wait_bounded(s_bar, 0, p.wait_polls);
        if (lane == 0) *s_flag = ok ? 1u : 0u;
    }
    __syncthreads();
    if (*s_flag == 0u) {
        // The wait ran out.  Nothing of the frame is written.  If the copy was issued it is still
        // on its way into this CTA's shared memory, so one warp keeps the CTA alive until it lands.
        if (tid == 0) atomicOr(p.status, kFlagTimeout);
        if (warp == 0 && !p.skip_staging) mbar_wait_bounded(s_bar, 0, kDrainPolls);
        return;
    }
    mbar_try_wait(s_bar, 0);              // completed phase: makes the staged bytes visible to this thread

    // ---- per-agent traversal set-up and box binning
    const int gx = p.gx, gz = p.gz;
    // voxel-index strides of the y-packed layout: x and z move by whole columns, y by single bits
    const int stride_x = 1 << p.lay.ysh, stride_z = gx << p.lay.ysh;
    // Traversal is confined to the cell box [lo, hi) that holds every filled voxel of this env
    // (nothing outside it can be hit), so rays that leave it, e.g. into the sky, stop there.
    const int lox = s_count[1], loy = s_count[2], loz = s_count[3];
    const int hix = s_count[4], hiy = s_count[5], hiz = s_count[6];
    const bool any_voxel = (lox < hix) && (loy < hiy) && (loz < hiz);
    const uint32_t occ_base = OCC_SHARED ? smem_addr(smem) : 0u;
    const uint32_t vi_bias = 8u * occ_base;
    const int P_ = p.palette;
    const uint32_t lut_base = smem_addr(s_lut);
    const uint32_t inside_row = lut_base + (uint32_t)(kFaceInside * P_ * 4);
    // position of cell (cx, cy, cz) in the walk's own terms (see MV_DDA_*)
    auto cell_pos = [&](int cx, int cy, int cz) -> uint32_t {
        return COLW ? occ_base + 4u * (uint32_t)(cx + gx * cz) : vi_bias + (uint32_t)(stride_x * cx + stride_z * cz + cy);
    };
    auto cell_filled = [&](int cx, int cy, int cz) -> bool {
        const uint32_t u = (uint32_t)(stride_x * cx + stride_z * cz + cy);
        return (s_occ[u >> 5] >> (u & 31)) & 1u;
    };
    for (int slot = tid; slot < kDdaVecs * apc; slot += NT) {
        // DDA start table of agent ag, entry 3*signs + axis (bit c of `signs` set: direction component c
        // negative): x = distance (>= 0) from the eye to the cell face the ray meets first, y = cells
        // left before the occupied box ends that way, z = what a step along the axis adds to the
        // position (column-word flavour: byte stride for x and z, rotate count for y), w = shared-memory
        // address of the colour-table row of the face entered by a step along this axis.
        const int ag = slot / kDdaVecs, e = slot - ag * kDdaVecs;
        const int signs = e / 3, ax = e - 3 * signs, neg = (signs >> ax) & 1;
        float4 *rec = agent_rec(ag);
        const float4 c0 = rec[0];
        const float Pc = ax == 0 ? c0.x : (ax == 1 ? c0.y : c0.z);
        const bool cam_in = any_voxel && (c0.x >= (float)lox) && (c0.x < (float)hix) && (c0.y >= (float)loy) &&
                            (c0.y < (float)hiy) && (c0.z >= (float)loz) && (c0.z < (float)hiz);
        int cx0 = 0, cy0 = 0, cz0 = 0;
        if (cam_in) { cx0 = (int)floorf(c0.x); cy0 = (int)floorf(c0.y); cz0 = (int)floorf(c0.z); }
        const int cc = ax == 0 ? cx0 : (ax == 1 ? cy0 : cz0);
        const int lo_c = ax == 0 ? lox : (ax == 1 ? loy : loz), hi_c = ax == 0 ? hix : (ax == 1 ? hiy : hiz);
        int st;
        if (COLW) st = ax == 0 ? (neg ? -4 : 4) : (ax == 1 ? (neg ? 31 : 1) : (neg ? -4 * gx : 4 * gx));
        else st = (ax == 0 ? stride_x : (ax == 1 ? 1 : stride_z)) * (neg ? -1 : 1);
        agent_dda(ag)[e] = make_float4(neg ? Pc - (float)cc : (float)(cc + 1) - Pc,
                                       neg ? (float)(cc - lo_c) : (float)(hi_c - 1 - cc), __int_as_float(st),
                                       __uint_as_float(lut_base + (uint32_t)((2 * ax + neg) * P_ * 4)));
        if (e == 0) {
            const bool filled = cam_in && cell_filled(cx0, cy0, cz0);
            rec[3].x = filled ? 0.0f : kInf;     // hit time a ray starts with: the eye's own voxel, or none yet
            rec[3].y = __uint_as_float(__float_as_uint(rec[3].y) | (cam_in ? kAgentInside : 0u) | (filled ? kAgentFilled : 0u));
            // exit-time factor: pulls the exit in by the rounding drift of the accumulated crossing
            // times; -inf (the product is then -inf or NaN and the first test ends the walk) when the
            // eye sits in a filled voxel
            rec[4] = make_float4(__uint_as_float(1u << cy0), filled ? -kInf : p.exit_scale,
                                 __uint_as_float(filled ? inside_row : kNoRow), __uint_as_float(cell_pos(cx0, cy0, cz0)));
            const unsigned long long mp = reinterpret_cast<unsigned long long>(
                p.mat + (size_t)env * ((size_t)gx * gz << p.lay.ysh) - vi_bias);
            rec[5] = make_float4(__uint_as_float((uint32_t)mp), __uint_as_float((uint32_t)(mp >> 32)),
                                 __uint_as_float(p.sky_rgbx), p.miss_depth);
        }
    }
    {
        const int nb = min(s_count[0], p.max_boxes);
        // (dealt from the last thread down, so that the warps that build the DDA tables above are not
        // the ones that bin the boxes)
        for (int i = NT - 1 - tid; i < apc * p.max_boxes; i += NT) {
            const int ag = i / p.max_boxes, b = i - ag * p.max_boxes;
            const float4 *rec = agent_rec(ag);
            const float4 c0 = rec[0], c1 = rec[1], c2 = rec[2];
            const float Px = c0.x, Py = c0.y, Pz = c0.z, Fx = c0.w, Fy = c1.x, Fz = c1.y;
            const float Rx = c1.z, Ry = c1.w, Rz = c2.x, Ux = c2.y, Uy = c2.z, Uz = c2.w;
            const int self_box = __float_as_int(rec[3].z);
            const float r2 = Rx * Rx + Ry * Ry + Rz * Rz, u2 = Ux * Ux + Uy * Uy + Uz * Uz;
            const float ir2 = 1.0f / r2, iu2 = 1.0f / u2;
            const float4 A = s_box[2 * b], B = s_box[2 * b + 1];
            const float lx = A.x - Px, ly = A.y - Py, lz = A.z - Pz;
            const float hx = A.w - Px, hy = B.x - Py, hz = B.y - Pz;
            const bool valid = (b < nb) && (b != self_box) && (A.x < A.w) && (A.y < B.x) && (A.z < B.y);
            float tmin = kInf, tmax = -kInf, fxmin = kInf, fxmax = -kInf, fymin = kInf, fymax = -kInf;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float vx = (c & 1) ? hx : lx, vy = (c & 2) ? hy : ly, vz = (c & 4) ? hz : lz;
                const float t = vx * Fx + vy * Fy + vz * Fz;
                const float u = (vx * Rx + vy * Ry + vz * Rz) * ir2;
                const float w = (vx * Ux + vy * Uy + vz * Uz) * iu2;
                tmin = fminf(tmin, t); tmax = fmaxf(tmax, t);
                const float it = 1.0f / fmaxf(t, 1e-3f);
                const float fx = (u * it + (float)(W - 1)) * 0.5f;     // pixel column of the projection
                const float fy = ((float)(H - 1) - w * it) * 0.5f;     // pixel row
                fxmin = fminf(fxmin, fx); fxmax = fmaxf(fxmax, fx);
                fymin = fminf(fymin, fy); fymax = fmaxf(fymax, fy);
            }
            const bool front = tmin > 0.05f;                 // whole box safely in front of the eye plane
            agent_rel(ag)[2 * b] = make_float4(lx, ly, lz, front ? tmin * 0.9999f : 0.0f);
            agent_rel(ag)[2 * b + 1] = make_float4(hx, hy, hz, B.z);
            if (!valid || tmax < -1e-3f) continue;           // ignored, or wholly behind the eye
            int px0 = 0, px1 = W - 1, py0 = 0, py1 = H - 1;
            if (front) {
                px0 = (int)ceilf(fmaxf(fxmin - 0.25f, 0.0f));
                px1 = (int)floorf(fminf(fxmax + 0.25f, (float)(W - 1)));
                py0 = (int)ceilf(fmaxf(fymin - 0.25f, 0.0f));
                py1 = (int)floorf(fminf(fymax + 0.25f, (float)(H - 1)));
                if (px0 > px1 || py0 > py1) continue;
            }
            const uint32_t bit = 1u << (b & 31);
            uint32_t *mask = agent_mask(ag);
            for (int ty = py0 >> 2; ty <= (py1 >> 2); ++ty)
                for (int tx = px0 >> 3; tx <= (px1 >> 3); ++tx)
                    {
                        uint32_t *tm = mask + (ty * p.tiles_x + tx) * ms;
                        atomicOr(tm + m0 + (b >> 5), bit);
                        if (mw > 1) atomicOr(tm, bit);          // the summary word only has to be non-zero
                    }
        }
    }
#if MV_BRICKS == 1
    unsigned char *s_brick = smem + p.smem_misc_off + 32;
    if (COLW) {
        const int bxn = gx >> 2, bzn = gz >> 2;
        for (int i = tid; i < bxn * bzn; i += NT) {
            const int bx = i % bxn, bz = i / bxn;
            uint32_t m = 0;
            for (int j = 0; j < 4; ++j)
                for (int k = 0; k < 4; ++k) m |= s_occ[(4 * bx + k) + gx * (4 * bz + j)];
            uint32_t byte = 0;
            for (int by = 0; by < 8; ++by) byte |= ((m >> (4 * by)) & 0xFu) ? (1u << by) : 0u;
            s_brick[i] = (unsigned char)byte;
        }
    }
#endif
    __syncthreads();

    const float flox = (float)lox, floy = (float)loy, floz = (float)loz;
    const float fhix = (float)hix, fhiy = (float)hiy, fhiz = (float)hiz;

    // ---- per-lane constants of the 8 x 4 tile: pixel offsets and the store plan.  Depth goes to the
    // lane's own pixel.  A tile row's RGB is 24 bytes = six 32-bit words; word j starts inside pixel
    // q = j + j/3 of the row (at its byte j % 3) and ends inside pixel q + 1, so the lanes of pixels
    // 0, 1, 2, 4, 5, 6 of each row write one word each, picked by a byte permute from the lane's own
    // packed colour and its right neighbour's; the lanes of pixels 3 and 7 store no RGB word.  keep()
    // pins the constants in registers: recomputing them per tile costs more issue slots than the
    // registers are worth.
    constexpr int kWarps = NT / 32;
    float lane_a = (float)(2 * (lane & 7)), lane_b = (float)(2 * (lane >> 3));
    const int st_r = lane >> 3, st_q = lane & 7, st_j = st_q - (st_q >> 2), st_byte = st_q & 3;
    // bytes st_byte.. of the own pixel (3 of them at most), then the neighbour's from its byte 0 (selector 4..)
    uint32_t st_sel = st_byte == 0 ? 0x4210u : (st_byte == 1 ? 0x5421u : (st_byte == 2 ? 0x6542u : 0xffffffffu));
    const int depth_lane_off = (lane >> 3) * W + (lane & 7);
    const int rgb_lane_off = st_r * W * 3 + st_j * 4;
    keep(lane_a); keep(lane_b); keep(st_sel);
    const uint32_t tile_begin = smem_addr(s_tile) + 16u * (uint32_t)warp;
#if MV_PROBE == 3
    uint32_t tile_end = smem_addr(s_tile);
#else
    uint32_t tile_end = smem_addr(s_tile) + 16u * (uint32_t)ntiles;
#endif
    uint32_t mask_step = 4u * kWarps * (uint32_t)ms;                        // bytes between a warp's consecutive tile masks
    keep(tile_end); keep(mask_step);

    for (int ag = 0; ag < apc; ++ag) {
        const int obs = obs0 + ag;
        uint8_t *rgb_obs = p.rgb + (size_t)obs * H * W * 3;
        float *depth_obs = p.depth + (size_t)obs * H * W;
        const float4 c0 = agent_rec(ag)[0], c3 = agent_rec(ag)[3];
        const uint32_t aflags = __float_as_uint(c3.y);
        if (aflags & kAgentBad) {                   // non-finite camera: a sky frame
            write_sky<NT>(rgb_obs, depth_obs, W * H, p.sky_rgbx, p.miss_depth);
            continue;
        }
        const float Px = c0.x, Py = c0.y, Pz = c0.z;
        const bool cam_in = (aflags & kAgentInside) != 0;
        const int ov_count = __float_as_int(c3.w);
        // non-zero: every tile takes the slow branch (an overlay that cannot flag its tiles in the box mask)
        uint32_t rare = (ov_count > 0 && p.max_boxes >= 32) ? 2u : 0u;
        keep(rare);
        uint32_t abase = smem_addr(agent_rec(ag));
        uint32_t mask_p = smem_addr(agent_mask(ag) + (size_t)warp * ms);
        // (store addresses as global-space addresses for the PTX store block)
        unsigned long long depth_lane = (unsigned long long)__cvta_generic_to_global(depth_obs + depth_lane_off);
        unsigned long long rgb_lane = (unsigned long long)__cvta_generic_to_global(rgb_obs + rgb_lane_off);
        keep(abase);
        asm volatile("" : "+l"(depth_lane), "+l"(rgb_lane));

        // ---- tiles: warp w takes tiles w, w + nwarps, ... (8 x 4 pixels, one per lane).  Two loops, so
        // that the choice between the common case and the rest is taken per agent, not per tile; what
        // follows the walk is the same for both.  The warp-wide reduction and shuffle in it name all 32
        // lanes, so they wait by themselves for lanes whose walk ran longer.
        auto finish_tile = [&](uint32_t tile_p, uint32_t mask_p, int tile_px, uint32_t pos, uint32_t bit, uint32_t row,
                               uint32_t sgn3, float t_hit, float dtx, float dty, float dtz) {
            // ---- the hit voxel's material byte is asked for from global memory (its colour is looked up
            // in the shaded table only in the store block, after everything that does not need it), this
            // tile's first box-mask word is read, and the latest voxel hit of the warp is found (boxes wholly
            // behind it are skipped).  Predicated, not branched; sky colour and miss depth ride with the
            // material store's address in the agent block.  (Column-word flavour: the voxel index is rebuilt from
            // the column's address and the bit.)
            uint32_t rgbx, m, mat_id;
            float depth, tb, wmax;
            {
                uint32_t vi = pos;
                if (COLW) {
                    uint32_t y;
                    asm("bfind.u32 %0, %1;" : "=r"(y) : "r"(bit));
                    vi = (pos << 3) + y;
                }
                asm volatile("{\n"
                    " .reg .pred pv;\n"
                    " .reg .b32 skyb, missb, tbb, wmb;\n"
                    " .reg .b64 mp, sm;\n"
                    " ld.shared.v2.b64 {mp, sm}, [%9+80];\n"
                    " ld.shared.u32 %2, [%10];\n"
                    " mov.b64 {skyb, missb}, sm;\n"
                    " mov.b32 %0, skyb;\n"
                    " mov.b32 %1, missb;\n"
                    " setp.ne.u32 pv, %6, 0xffffffff;\n"
                    " mad.wide.u32 mp, %7, 1, mp;\n"
                    " mov.b32 tbb, %8;\n"
                    " @pv ld.global.nc.u8 %5, [mp];\n"
                    " redux.sync.max.u32 wmb, tbb, 0xffffffff;\n"
                    " mov.b32 %3, tbb;\n"
                    " mov.b32 %4, wmb;\n"
                    " @pv mov.f32 %1, %8;\n"
                    "}\n"
                    : "=&r"(rgbx), "=&f"(depth), "=&r"(m), "=&f"(tb), "=&f"(wmax), "=&r"(mat_id)
                    : "r"(row), "r"(vi), "f"(t_hit), "r"(abase), "r"(mask_p)
                    : "memory");
            }
#if MV_PROBE == 9
            depth = t_hit;
#endif
#if MV_PROBE >= 2 && MV_PROBE < 9
            m = 0;
#endif

            // ---- the less common work, behind one test: boxes binned to this tile (or more than 32 boxes
            // per environment) and the GUI overlay.  A box wins only with a strictly smaller time.
            if ((m | rare) != 0u) {
                if (p.max_boxes < 32) m &= ~kOverlayTileBit;
                if (m != 0u) {
                    // (more than 32 boxes per env: m was the summary; start with the first real word)
                    if (mw > 1) asm volatile("ld.shared.u32 %0, [%1+4];" : "=r"(m) : "r"(mask_p));
                    // signed reciprocals again, and the ray's rows of the DDA table for the faces
                    const float ix = __uint_as_float(__float_as_uint(dtx) | (sgn3 << 31));
                    const float iy = __uint_as_float(__float_as_uint(dty) | ((sgn3 & 2u) << 30));
                    const float iz = __uint_as_float(__float_as_uint(dtz) | ((sgn3 & 4u) << 29));
                    const uint32_t tab = abase + 48u * sgn3;
                    uint32_t baddr = 0;
                    for (int w = 0;;) {
                        while (m) {
                            const int b = (__ffs(m) - 1) + 32 * w;
                            m &= m - 1;
                            float4 lo, hi;
                            const uint32_t rel_p = abase + kAgentRelOff + 32u * (uint32_t)b;
                            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(lo.x), "=f"(lo.y), "=f"(lo.z), "=f"(lo.w) : "r"(rel_p));
                            if (lo.w > wmax) continue;
                            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4+16];" : "=f"(hi.x), "=f"(hi.y), "=f"(hi.z), "=f"(hi.w) : "r"(rel_p));
                            const float x1 = lo.x * ix, x2 = hi.x * ix, y1 = lo.y * iy, y2 = hi.y * iy;
                            const float z1 = lo.z * iz, z2 = hi.z * iz;
                            const float nx = fminf(x1, x2), ny = fminf(y1, y2), nz = fminf(z1, z2);
                            const float tn = max3f(nx, ny, nz);
                            const float tf = min3f(fmaxf(x1, x2), fmaxf(y1, y2), fmaxf(z1, z2));
                            const float t = fmaxf(tn, 0.0f);
                            if ((tn <= tf) && (tf > 0.0f) && (t < tb)) {
                                tb = t;
                                uint32_t r = inside_row;
                                if (!(tn < 0.0f))
                                    asm volatile("ld.shared.u32 %0, [%1+" MV_TAB_ROW "];" : "=r"(r)
                                                 : "r"(tab + ((nx == tn) ? 0u : ((ny == tn) ? 16u : 32u))));
                                baddr = r + 4u * __float_as_uint(hi.w);
                            }
                        }
                        if (++w >= mw) break;
                        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(m) : "r"(mask_p + 4u * (uint32_t)(w + m0)));
                    }
                    if (baddr) {
                        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(rgbx) : "r"(baddr));
                        depth = tb + 0.0f;
                        row = kNoRow;                            // the voxel behind the box is not looked up
                    }
                }
                // GUI overlay: rectangles in list order, later ones on top; depth is left alone
                if (ov_count > 0) {
                    const uint32_t tile_no = (tile_p - smem_addr(s_tile)) >> 4;
                    if ((agent_ovtile(ag)[tile_no >> 5] >> (tile_no & 31)) & 1u) {
                        const int4 *ov = agent_ov(ag);
                        const int px = (tile_px % W) + (lane & 7), py = (tile_px / W) + (lane >> 3);
                        if (row != kNoRow) {                     // the rectangles go over the voxel colour: look it up now
                            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(rgbx) : "r"(row + 4u * mat_id));
                            row = kNoRow;
                        }
                        for (int r = 0; r < ov_count; ++r) {
                            const int4 q = ov[2 * r];
                            if (px >= q.x && px < q.z && py >= q.y && py < q.w) rgbx = (uint32_t)ov[2 * r + 1].x;
                        }
                    }
                }
            }

            // ---- store: depth rows are 32-byte segments; RGB rows are 24 bytes = 6 packed words
            asm volatile("{\n"
                " .reg .pred ps, pv;\n"
                " .reg .b32 ca, cb, cc;\n"
                " .reg .b64 ad;\n"
                " mad.wide.s32 ad, %2, 4, %3;\n"
                " st.global.f32 [ad], %1;\n"
                " setp.ne.u32 pv, %6, 0xffffffff;\n"
                " mad.lo.u32 ca, %7, 4, %6;\n"
                " mov.b32 cc, %0;\n"
                " @pv ld.shared.u32 cc, [ca];\n"
                " shfl.sync.down.b32 cb, cc, 1, 31, 0xffffffff;\n"
                " mad.wide.s32 ad, %2, 3, %4;\n"
                " prmt.b32 ca, cc, cb, %5;\n"
                " setp.ge.s32 ps, %5, 0;\n"
                " @ps st.global.u32 [ad], ca;\n"
                "}\n"
                :: "r"(rgbx), "f"(depth), "r"(tile_px), "l"(depth_lane), "l"(rgb_lane), "r"(st_sel), "r"(row), "r"(mat_id)
                : "memory");
        };
        if (COLW && cam_in && !MV_BRICKS) {
            for (uint32_t tile_p = tile_begin; tile_p < tile_end; tile_p += 16u * kWarps, mask_p += mask_step) {
                int tile_px;
                uint32_t pos, bit = 0, row, sgn3;
                float t_hit, dtx, dty, dtz;
                // ---- the common case in one block of PTX: tile record, ray through the pixel centre
                // (d = F + a*Rs + b*Us, a = 2px+1-W, b = H-1-2py, two chained FMAs per component),
                // reciprocals, the DDA table rows for the ray's signs
                // {distance to the first face, cells left, step, colour row} per axis, first crossing
                // times, exit time, then the walk.  The basis is re-read from shared memory per tile:
                // three broadcast loads cost less than nine registers held across the walk.
                // A direction component that is exactly zero needs no special case here: its reciprocal
                // is +-inf, so its crossing time is +inf (or NaN when the eye sits exactly on the face,
                // which min and the compares ignore) and that axis is never stepped, which is the rule
                // for such rays; the exit time ignores the axis the same way.
                asm volatile("{\n"
                    MV_DDA_DECL
                    " .reg .f32 Ta, Tb, Fx, Fy, Fz, Rx, Ry, Rz, Ux, Uy, Uz, ca, cb, dx, dy, dz, ix, iy, iz;\n"
                    " .reg .f32 q0, q1, q2, q3, q4, q5, esc;\n"
                    " .reg .b32 u, tab;\n"
                    " ld.shared.v4.b32 {Ta, Tb, %0, _}, [%9];\n"
                    " ld.shared.f32 Fx, [%10+12];\n"
                    " ld.shared.v4.f32 {Fy, Fz, Rx, Ry}, [%10+16];\n"
                    " ld.shared.v4.f32 {Rz, Ux, Uy, Uz}, [%10+32];\n"
                    " ld.shared.v4.b32 {bit, esc, %4, pos}, [%10+64];\n"
                    " add.f32 ca, Ta, %11;\n"
                    " sub.f32 cb, Tb, %12;\n"
                    " fma.rn.f32 dx, ca, Rx, Fx;\n"
                    " fma.rn.f32 dy, ca, Ry, Fy;\n"
                    " fma.rn.f32 dz, ca, Rz, Fz;\n"
                    " fma.rn.f32 dx, cb, Ux, dx;\n"
                    " fma.rn.f32 dy, cb, Uy, dy;\n"
                    " fma.rn.f32 dz, cb, Uz, dz;\n"
                    " abs.f32 ix, dx;\n"
                    " abs.f32 iy, dy;\n"
                    " abs.f32 iz, dz;\n"
                    " rcp.approx.ftz.f32 dtx, ix;\n"
                    " rcp.approx.ftz.f32 dty, iy;\n"
                    " rcp.approx.ftz.f32 dtz, iz;\n"
                    " mov.b32 u, dx;\n"
                    " shr.u32 %8, u, 31;\n"
                    " mov.b32 u, dy;\n"
                    " shr.u32 u, u, 30;\n"
                    " lop3.b32 %8, u, 2, %8, 0xEA;\n"
                    " mov.b32 u, dz;\n"
                    " shr.u32 u, u, 29;\n"
                    " lop3.b32 %8, u, 4, %8, 0xEA;\n"
                    " mad.lo.u32 tab, %8, 48, %10;\n"
                    " ld.shared.v4.b32 {q0, q1, sx, _}, [tab+" MV_TAB_X "];\n"
                    " ld.shared.v4.b32 {q2, q3, sy, _}, [tab+" MV_TAB_Y "];\n"
                    " ld.shared.v4.b32 {q4, q5, sz, _}, [tab+" MV_TAB_Z "];\n"
                    " mul.f32 tx, q0, dtx;\n"
                    " mul.f32 ty, q2, dty;\n"
                    " mul.f32 tz, q4, dtz;\n"
                    " fma.rn.f32 q1, q1, dtx, tx;\n"
                    " fma.rn.f32 q3, q3, dty, ty;\n"
                    " fma.rn.f32 q5, q5, dtz, tz;\n"
                    " min.f32 q1, q1, q3, q5;\n"
                    " mul.f32 texit, q1, esc;\n"
#if MV_PROBE >= 1 && MV_PROBE < 9
                    " mov.f32 texit, 0fFF800000;\n"
#endif
                    " ld.shared.f32 thit, [%10+48];\n"
                    " mov.s32 it, " MV_STEP_BUDGET ";\n"
                    MV_DDA_LOOP(MV_DDA_STEP_COLW)
                    " @py add.u32 tab, tab, 16;\n"
                    " @pz add.u32 tab, tab, 32;\n"
                    " @ph ld.shared.u32 %4, [tab+" MV_TAB_ROW "];\n"
#if MV_PROBE == 9
                    " mov.f32 thit, ns;\n"
#endif
                    " mov.b32 %1, pos;\n"
                    " mov.b32 %2, bit;\n"
                    " mov.f32 %3, thit;\n"
                    " mov.f32 %5, dtx;\n"
                    " mov.f32 %6, dty;\n"
                    " mov.f32 %7, dtz;\n"
                    "}\n"
                    : "=&r"(tile_px), "=&r"(pos), "=&r"(bit), "=&f"(t_hit), "=&r"(row), "=&f"(dtx), "=&f"(dty), "=&f"(dtz), "=&r"(sgn3)
                    : "r"(tile_p), "r"(abase), "f"(lane_a), "f"(lane_b)
                    : "memory");
                finish_tile(tile_p, mask_p, tile_px, pos, bit, row, sgn3, t_hit, dtx, dty, dtz);
            }
        } else {
            for (uint32_t tile_p = tile_begin; tile_p < tile_end; tile_p += 16u * kWarps, mask_p += mask_step) {
                int tile_px;
                uint32_t pos, bit = 0, row, sgn3;
                float t_hit, dtx, dty, dtz;
                // ---- every other case: the same steps in C++, with the eye possibly outside the
                // occupied box and either flavour of the walk
                float Ta, Tb;
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, _}, [%3];" : "=f"(Ta), "=f"(Tb), "=r"(tile_px) : "r"(tile_p));
                float Fx, Fy, Fz, Rx, Ry, Rz, Ux, Uy, Uz, esc;
                uint32_t pos0, row0, bit0;
                asm volatile("ld.shared.f32 %0, [%1+12];" : "=f"(Fx) : "r"(abase));
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4+16];" : "=f"(Fy), "=f"(Fz), "=f"(Rx), "=f"(Ry) : "r"(abase));
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4+32];" : "=f"(Rz), "=f"(Ux), "=f"(Uy), "=f"(Uz) : "r"(abase));
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4+64];" : "=r"(bit0), "=f"(esc), "=r"(row0), "=r"(pos0) : "r"(abase));
                const float a = Ta + lane_a, bb = Tb - lane_b;
                float dx = fmaf(bb, Ux, fmaf(a, Rx, Fx));
                float dy = fmaf(bb, Uy, fmaf(a, Ry, Fy));
                float dz = fmaf(bb, Uz, fmaf(a, Rz, Fz));
                dx = dx == 0.0f ? 1e-30f : dx;
                dy = dy == 0.0f ? 1e-30f : dy;
                dz = dz == 0.0f ? 1e-30f : dz;
                const float ix = fast_rcp(dx), iy = fast_rcp(dy), iz = fast_rcp(dz);
                dtx = fabsf(ix); dty = fabsf(iy); dtz = fabsf(iz);
                sgn3 = (__float_as_uint(dx) >> 31) | ((__float_as_uint(dy) >> 30) & 2u) | ((__float_as_uint(dz) >> 29) & 4u);
                const uint32_t tab = abase + 48u * sgn3;
                float qxx, qxy, qyx, qyy, qzx, qzy;
                int sx, sy, sz;
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, _}, [%3+" MV_TAB_X "];" : "=f"(qxx), "=f"(qxy), "=r"(sx) : "r"(tab));
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, _}, [%3+" MV_TAB_Y "];" : "=f"(qyx), "=f"(qyy), "=r"(sy) : "r"(tab));
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, _}, [%3+" MV_TAB_Z "];" : "=f"(qzx), "=f"(qzy), "=r"(sz) : "r"(tab));
                float t0x, t0y, t0z, t_exit;
                t_hit = 0.0f;
                pos = pos0; bit = bit0; row = row0;
                if (cam_in) {
                    t0x = qxx * dtx;
                    t0y = qyx * dty;
                    t0z = qzx * dtz;
                    t_exit = min3f(fmaf(qxy, dtx, t0x), fmaf(qyy, dty, t0y), fmaf(qzy, dtz, t0z)) * esc;
                } else {
                    // eye outside the occupied box: clip the ray to it, start in the entry cell
                    const bool ngx = dx < 0.0f, ngy = dy < 0.0f, ngz = dz < 0.0f;
                    const float x1 = (flox - Px) * ix, x2 = (fhix - Px) * ix;
                    const float y1 = (floy - Py) * iy, y2 = (fhiy - Py) * iy;
                    const float z1 = (floz - Pz) * iz, z2 = (fhiz - Pz) * iz;
                    const float nrx = fminf(x1, x2), nry = fminf(y1, y2), nrz = fminf(z1, z2);
                    const float tn = max3f(nrx, nry, nrz);
                    const float tf = min3f(fmaxf(x1, x2), fmaxf(y1, y2), fmaxf(z1, z2));
                    const bool alive = any_voxel && (tn <= tf) && (tf > 0.0f);
                    const int eaxis = tn < 0.0f ? -1 : (nrx == tn ? 0 : (nry == tn ? 1 : 2));
                    t_hit = alive ? fmaxf(tn, 0.0f) : 0.0f;
                    int cx = min(max((int)floorf(fmaf(t_hit, dx, Px)), lox), hix - 1);
                    int cy = min(max((int)floorf(fmaf(t_hit, dy, Py)), loy), hiy - 1);
                    int cz = min(max((int)floorf(fmaf(t_hit, dz, Pz)), loz), hiz - 1);
                    if (eaxis == 0) cx = ngx ? hix - 1 : lox;
                    if (eaxis == 1) cy = ngy ? hiy - 1 : loy;
                    if (eaxis == 2) cz = ngz ? hiz - 1 : loz;
                    if (!alive) { cx = cy = cz = 0; }
                    pos = cell_pos(cx, cy, cz);
                    bit = 1u << cy;
                    t0x = ((float)(cx + (ngx ? 0 : 1)) - Px) * ix;
                    t0y = ((float)(cy + (ngy ? 0 : 1)) - Py) * iy;
                    t0z = ((float)(cz + (ngz ? 0 : 1)) - Pz) * iz;
                    t_exit = min3f(fmaf(ngx ? (float)(cx - lox) : (float)(hix - 1 - cx), dtx, t0x),
                                   fmaf(ngy ? (float)(cy - loy) : (float)(hiy - 1 - cy), dty, t0y),
                                   fmaf(ngz ? (float)(cz - loz) : (float)(hiz - 1 - cz), dtz, t0z)) * p.exit_scale;
                    const bool filled = alive && cell_filled(cx, cy, cz);
                    // entered through the box face of axis eaxis, or the eye is inside a solid
                    if (filled) {
                        if (eaxis < 0) row = inside_row;
                        else asm volatile("ld.shared.u32 %0, [%1+" MV_TAB_ROW "];" : "=r"(row) : "r"(tab + 16u * (uint32_t)eaxis));
                    }
                    if (!alive || filled) t_exit = -kInf;
                }
#if MV_PROBE >= 1 && MV_PROBE < 9
                t_exit = -kInf;
#endif
#define MV_DDA_IO                                                                                         \
                    : "+r"(pos), "+r"(bit), "+f"(t_hit), "+r"(row)                                                  \
                    : "f"(t0x), "f"(t0y), "f"(t0z), "f"(dtx), "f"(dty), "f"(dtz), "r"(sx), "r"(sy), "r"(sz), "f"(t_exit), \
                      "r"(p.max_steps), "r"(tab), "l"(s_occ)                                                       \
                    : "memory"
#define MV_DDA_IN                                                                                         \
                    " mov.b32 pos, %0;\n mov.b32 bit, %1;\n mov.f32 thit, %2;\n"                                    \
                    " mov.f32 tx, %4;\n mov.f32 ty, %5;\n mov.f32 tz, %6;\n mov.f32 dtx, %7;\n mov.f32 dty, %8;\n"   \
                    " mov.f32 dtz, %9;\n mov.b32 sx, %10;\n mov.b32 sy, %11;\n mov.b32 sz, %12;\n mov.f32 texit, %13;\n" \
                    " mov.s32 it, " MV_STEP_BUDGET ";\n mov.b64 gbase, %16;\n"
#define MV_DDA_OUTS                                                                                       \
                    " selp.u32 a, 16, 32, py;\n selp.u32 a, 0, a, px;\n add.u32 a, a, %15;\n"                        \
                    " @ph ld.shared.u32 %3, [a+" MV_TAB_ROW "];\n mov.b32 %0, pos;\n mov.b32 %1, bit;\n mov.f32 %2, thit;\n"
#if MV_BRICKS == 1
                if (COLW && cam_in) {
                    // two-level traversal: per brick, its exit time; occupied bricks are walked by the PTX
                    // loop up to that time, then every axis is advanced past its crossings up to it (one
                    // crossing after a walked brick, several across an empty one) and the arrival cell tested
                    const int lgx = 31 - __clz(gx);
                    const float adx = fabsf(dx), ady = fabsf(dy), adz = fabsf(dz);
                    const float t_exit_all = t_exit;
                    for (int guard = 0; guard < 3 * 256 + 8 && row == kNoRow; ++guard) {
                        const uint32_t col = (pos - occ_base) >> 2;
                        const int cx = (int)(col & (uint32_t)(gx - 1)), cz = (int)(col >> lgx), cy = 31 - __clz(bit);
                        const int nbx = (sgn3 & 1u) ? (cx & 3) : 3 - (cx & 3), nby = (sgn3 & 2u) ? (cy & 3) : 3 - (cy & 3);
                        const int nbz = (sgn3 & 4u) ? (cz & 3) : 3 - (cz & 3);
                        const float tbk = min3f(fmaf((float)nbx, dtx, t0x), fmaf((float)nby, dty, t0y), fmaf((float)nbz, dtz, t0z));
                        if ((s_brick[(cx >> 2) + (gx >> 2) * (cz >> 2)] >> (cy >> 2)) & 1u) {
                            t_exit = fminf(tbk, t_exit_all);
                            asm volatile("{\n" MV_DDA_DECL MV_DDA_IN MV_DDA_LOOP(MV_DDA_STEP_COLW) MV_DDA_OUTS
                                         " mov.f32 %4, tx;\n mov.f32 %5, ty;\n mov.f32 %6, tz;\n}\n"
                                         : "+r"(pos), "+r"(bit), "+f"(t_hit), "+r"(row), "+f"(t0x), "+f"(t0y), "+f"(t0z)
                                         : "f"(dtx), "f"(dty), "f"(dtz), "r"(sx), "r"(sy), "r"(sz), "f"(t_exit), "r"(p.max_steps),
                                           "r"(tab), "l"(s_occ)
                                         : "memory");
                            if (row != kNoRow) break;
                        }
                        if (tbk >= t_exit_all) break;
                        // crossings of each axis up to the brick's exit time (with a tolerance: the exit
                        // time is a product, the crossing times are sums)
                        const float tol = fmaf(tbk, 1e-5f, 1e-6f);
                        const int mx = t0x <= tbk + tol ? (int)floorf(fmaxf(tbk - t0x, 0.0f) * adx + 1e-3f) + 1 : 0;
                        const int my = t0y <= tbk + tol ? (int)floorf(fmaxf(tbk - t0y, 0.0f) * ady + 1e-3f) + 1 : 0;
                        const int mz = t0z <= tbk + tol ? (int)floorf(fmaxf(tbk - t0z, 0.0f) * adz + 1e-3f) + 1 : 0;
                        // nothing to cross: the walk itself took the step out of the brick (its crossing times are
                        // sums, the brick's exit time a product); look at the new brick
                        if (mx + my + mz == 0) continue;
                        // never past the occupied cell box (integer test, so the position stays valid)
                        const int rx = (sgn3 & 1u) ? cx - lox : hix - 1 - cx, ry = (sgn3 & 2u) ? cy - loy : hiy - 1 - cy;
                        const int rz = (sgn3 & 4u) ? cz - loz : hiz - 1 - cz;
                        if (mx > rx || my > ry || mz > rz) break;
                        t0x = fmaf((float)mx, dtx, t0x); t0y = fmaf((float)my, dty, t0y); t0z = fmaf((float)mz, dtz, t0z);
                        pos += (uint32_t)(mx * sx + mz * sz);
                        bit = __funnelshift_l(bit, bit, (uint32_t)(my * sy) & 31u);
                        if (pos - occ_base >= p.lay.occ_bytes) break;        // (cannot happen; guards the load below)
                        uint32_t w;
                        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w) : "r"(pos));
                        if (w & bit) {
                            t_hit = tbk;
                            const float lastx = t0x - dtx, lasty = t0y - dty, lastz = t0z - dtz;     // the latest crossing taken
                            const float lx_ = mx ? lastx : -kInf, ly_ = my ? lasty : -kInf, lz_ = mz ? lastz : -kInf;
                            const float latest = fmaxf(lx_, fmaxf(ly_, lz_));
                            asm volatile("ld.shared.u32 %0, [%1+" MV_TAB_ROW "];" : "=r"(row)
                                         : "r"(tab + (lx_ == latest ? 0u : (ly_ == latest ? 16u : 32u))));
                        }
                    }
                } else
#endif
                if constexpr (COLW) {
                    asm volatile("{\n" MV_DDA_DECL MV_DDA_IN MV_DDA_LOOP(MV_DDA_STEP_COLW) MV_DDA_OUTS "}\n" MV_DDA_IO);
                } else if constexpr (OCC_SHARED) {
                    asm volatile("{\n" MV_DDA_DECL MV_DDA_IN MV_DDA_LOOP(MV_DDA_STEP_IDX) MV_DDA_OUTS "}\n" MV_DDA_IO);
                } else {
                    asm volatile("{\n" MV_DDA_DECL MV_DDA_IN MV_DDA_LOOP(MV_DDA_STEP_IDX_GLOBAL) MV_DDA_OUTS "}\n" MV_DDA_IO);
                }
#undef MV_DDA_IO
#undef MV_DDA_IN
#undef MV_DDA_OUTS
#if MV_PROBE != 9
                if (row == kNoRow) t_hit = kInf;          // no voxel hit
#endif
                finish_tile(tile_p, mask_p, tile_px, pos, bit, row, sgn3, t_hit, dtx, dty, dtz);
            }
        }
    }
}

}  // namespace mv
