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
// lane owns one pixel of the tile: it walks the occupancy grid with a branch-free 3D-DDA in
// shared memory, tests the tile's candidate boxes with slab tests, looks the colour up in the
// shaded table and the warp writes 24-byte RGB row segments as packed 32-bit words and 32-byte
// depth row segments.
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

// The DDA loop (see render_kernel).  Operands: %0 voxel index (in/out), %1 hit time (in/out: kept
// unless a filled cell is entered), %2 = shared-memory address of the colour-table row of the face
// entered at a hit (in/out, kept likewise), %3..%5 = crossing times per axis (in/out), %6..%8 = dt per
// axis, %9..%11 = index strides, %12 = exit time, %13 = step budget, %14 = shared-memory
// address of the ray's DDA table rows (whose fourth words are the colour-table rows per axis),
// %15 = 64-bit global base of the occupancy words (only when they are not staged in shared memory).
// One step: t = min(tx,ty,tz); leave when t >= exit time or when the cell entered by the previous step
// is filled (one branch for both); else the axis whose crossing time equals t (ties: x, then y, then
// z) advances: crossing time += dt, voxel index += stride; then the new cell's occupancy bit is
// tested.  Two registers alternate as t, so that after a hit the time at which the filled cell was
// entered is still there.  The voxel index carries 8x the shared-memory byte address of the occupancy
// grid, so (index >> 3) & ~3 is the word's address and index & 31 the bit (the index is
// ((x + grid_x*z) << ysh) | y: steps along x and z change the word, steps along y the bit).
#if defined(MV_PROBE) && MV_PROBE == 9
#define MV_DDA_COUNT " add.f32 ns, ns, 0f3F800000;\n"
#define MV_DDA_COUNT_OUT " mov.f32 %1, ns;\n"
#else
#define MV_DDA_COUNT
#define MV_DDA_COUNT_OUT
#endif
#define MV_DDA_ADVANCE(T, OUT)                       \
    " min.f32 " T ", %3, %4, %5;\n"                  \
    " setp.geu.or.f32 pq, " T ", %12, ph;\n"         \
    " @pq bra " OUT ";\n"                            \
    MV_DDA_COUNT                                     \
    " setp.eq.f32 px, %3, " T ";\n"                  \
    " setp.eq.and.f32 py|pz, %4, " T ", !px;\n"      \
    " @px add.f32 %3, %3, %6;\n"                     \
    " @px add.s32 %0, %0, %9;\n"                     \
    " @py add.f32 %4, %4, %7;\n"                     \
    " @py add.s32 %0, %0, %10;\n"                    \
    " @pz add.f32 %5, %5, %8;\n"                     \
    " @pz add.s32 %0, %0, %11;\n"
#define MV_DDA_TEST                                  \
    " shf.r.wrap.b32 w, w, 0, %0;\n"                 \
    " and.b32 w, w, 1;\n"                            \
    " setp.ne.u32 ph, w, 0;\n"
#define MV_DDA_LOAD_SHARED " shr.u32 a, %0, 3;\n and.b32 a, a, 0xfffffffc;\n ld.shared.u32 w, [a];\n"
#define MV_DDA_LOAD_GLOBAL " shr.u32 a, %0, 5;\n mad.wide.u32 ag, a, 4, %15;\n ld.global.nc.u32 w, [ag];\n"
#define MV_DDA_STEP(T, OUT) MV_DDA_ADVANCE(T, OUT) MV_DDA_LOAD_SHARED MV_DDA_TEST
#define MV_DDA_STEP_GLOBAL(T, OUT) MV_DDA_ADVANCE(T, OUT) MV_DDA_LOAD_GLOBAL MV_DDA_TEST
#define MV_DDA_PROLOGUE                              \
    "{\n"                                            \
    " .reg .pred px, py, pz, pq, ph;\n"              \
    " .reg .f32 ta, tb, ns;\n"                       \
    " .reg .u32 w, a;\n"                             \
    " .reg .u64 ag;\n"                               \
    " .reg .s32 it;\n"                               \
    " mov.s32 it, %13;\n"                            \
    " mov.f32 ns, 0f00000000;\n"                     \
    " mov.f32 tb, 0f00000000;\n"                     \
    " setp.ne.u32 ph, 0, 0;\n"                       \
    " setp.ne.u32 px, 0, 0;\n"                       \
    " setp.ne.u32 py, 0, 0;\n"                       \
    "MV_DDA_LOOP:\n"
#define MV_DDA_EPILOGUE                              \
    " sub.s32 it, it, 4;\n"                          \
    " setp.gt.s32 pq, it, 0;\n"                     \
    " @pq bra MV_DDA_LOOP;\n"                        \
    "MV_DDA_OUT_A:\n"                                \
    " @ph mov.f32 %1, tb;\n"                         \
    " bra MV_DDA_OUT;\n"                             \
    "MV_DDA_OUT_B:\n"                                \
    " @ph mov.f32 %1, ta;\n"                         \
    "MV_DDA_OUT:\n"                                  \
    " selp.u32 a, 16, 32, py;\n"                     \
    " selp.u32 a, 0, a, px;\n"                       \
    " add.u32 a, a, %14;\n"                          \
    " @ph ld.shared.u32 %2, [a+12];\n"               \
    MV_DDA_COUNT_OUT                                 \
    "}\n"
#define MV_DDA_BODY MV_DDA_PROLOGUE MV_DDA_STEP("ta", "MV_DDA_OUT_A") MV_DDA_STEP("tb", "MV_DDA_OUT_B") \
    MV_DDA_STEP("ta", "MV_DDA_OUT_A") MV_DDA_STEP("tb", "MV_DDA_OUT_B") MV_DDA_EPILOGUE
#define MV_DDA_BODY_GLOBAL MV_DDA_PROLOGUE MV_DDA_STEP_GLOBAL("ta", "MV_DDA_OUT_A") MV_DDA_STEP_GLOBAL("tb", "MV_DDA_OUT_B") \
    MV_DDA_STEP_GLOBAL("ta", "MV_DDA_OUT_A") MV_DDA_STEP_GLOBAL("tb", "MV_DDA_OUT_B") MV_DDA_EPILOGUE

#ifndef MV_PROBE
#define MV_PROBE 0
#endif
#ifndef MV_MINB
#define MV_MINB 3
#endif

constexpr uint32_t kAgentInside = 1u;      // eye inside the occupied cell box
constexpr uint32_t kAgentBad = 2u;         // non-finite camera: sky frame
constexpr int kAgentRecVecs = 4;           // float4 slots per agent: camera (3) + {start index, flags, self box, overlay count}
constexpr int kDdaVecs = 24;               // float4 slots per agent: 8 sign combinations x 3 axes

// OCC_SHARED: the occupancy bits are staged in shared memory with the rest of the env block (the
// normal case); otherwise only the block's tail (colour table, boxes, bounds) is staged and the
// occupancy is read from global memory through the read-only path.
template <int NT, bool OCC_SHARED>
__global__ void __launch_bounds__(NT, MV_MINB) render_kernel(const RenderParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int apc = p.agents_per_cta;
    const int obs0 = p.obs_begin + blockIdx.x * apc;
    const int env = obs0 / p.agents;
    const int W = p.W, H = p.H;
    const int ntiles = p.tiles_x * p.tiles_y;
    const int mw = p.mask_words;

    // bytes of the env block that are NOT staged (the occupancy, when it stays in global memory)
    const uint32_t unstaged = OCC_SHARED ? 0u : p.lay.occ_bytes;
    const unsigned char *env_block = p.env_blocks + (size_t)env * p.lay.stride;
    const uint32_t *s_occ = OCC_SHARED ? reinterpret_cast<const uint32_t *>(smem)
                                       : reinterpret_cast<const uint32_t *>(env_block);
    const unsigned char *s_lut = smem + (p.lay.lut_off - unstaged);
    const float4 *s_box = reinterpret_cast<const float4 *>(smem + (p.lay.box_off - unstaged));
    const int *s_count = reinterpret_cast<const int *>(smem + (p.lay.count_off - unstaged));
    float4 *s_tile = reinterpret_cast<float4 *>(smem + p.smem_tile_off);
    uint32_t *s_mask = reinterpret_cast<uint32_t *>(smem + p.smem_mask_off);
    float4 *s_rel = reinterpret_cast<float4 *>(smem + p.smem_rel_off);
    float4 *s_agent = reinterpret_cast<float4 *>(smem + p.smem_agent_off);
    float4 *s_dda = s_agent + apc * kAgentRecVecs;
    uint64_t *s_bar = reinterpret_cast<uint64_t *>(smem + p.smem_misc_off);
    uint32_t *s_flag = reinterpret_cast<uint32_t *>(smem + p.smem_misc_off + 8);
    int4 *s_ov = reinterpret_cast<int4 *>(smem + p.smem_ov_off);
    const int ov_slots = 2 * max(p.max_overlay, 1);                 // int4 slots per agent
    const int ovt_words = (ntiles + 31) / 32;
    uint32_t *s_ovtile = reinterpret_cast<uint32_t *>(s_ov + apc * ov_slots);

    // ---- stage the environment block
    if (tid == 0) mbar_init(s_bar, 1);
    __syncthreads();
    if (tid == 0 && !p.skip_staging) {
        mbar_expect_tx(s_bar, p.lay.block_bytes - unstaged);
        bulk_load(smem, env_block + unstaged, p.lay.block_bytes - unstaged, s_bar);
    }
    // ---- meanwhile: tile table, cleared masks, camera records, GUI rectangles
    for (int i = tid; i < apc * ntiles * mw; i += NT) s_mask[i] = 0u;
    for (int i = tid; i < ntiles; i += NT) {
        const int ty = i / p.tiles_x, tx = i - ty * p.tiles_x;
        // a = 2px+1-W and b = H-1-2py of the tile's first pixel (small integers: exact as floats)
        s_tile[i] = make_float4((float)(16 * tx + 1 - W), (float)(H - 1 - 8 * ty), __int_as_float(ty * 4 * W + tx * 8),
                                __int_as_float(i));
    }
    if (tid < apc) {
        const float4 *cq = reinterpret_cast<const float4 *>(p.cams + obs0 + tid);
        const float4 c3 = __ldg(cq + 3);
        s_agent[kAgentRecVecs * tid + 0] = __ldg(cq);
        s_agent[kAgentRecVecs * tid + 1] = __ldg(cq + 1);
        s_agent[kAgentRecVecs * tid + 2] = __ldg(cq + 2);
        const int ovc = p.overlay ? min(max(__ldg(p.overlay_count + obs0 + tid), 0), p.max_overlay) : 0;
        // slot 3: {start voxel index (filled in below), flags, self box, overlay count}
        s_agent[kAgentRecVecs * tid + 3] = make_float4(0.0f, __uint_as_float((__float_as_uint(c3.y) & kFlagBadCamera) ? kAgentBad : 0u),
                                                        c3.x, __int_as_float(ovc));
    }
    if (p.overlay) {
        // GUI rectangles of each observation (unpacked to x0,y0,x1,y1 / colour in two slots) and one
        // bit per tile that any rectangle touches, so untouched tiles pay a single bit test
        for (int i = tid; i < apc * ovt_words; i += NT) s_ovtile[i] = 0u;
        __syncthreads();
        for (int i = tid; i < apc * p.max_overlay; i += NT) {
            const int ag = i / p.max_overlay, r = i - ag * p.max_overlay;
            const int ovc = min(max(__ldg(p.overlay_count + obs0 + ag), 0), p.max_overlay);
            if (r >= ovc) continue;
            const int4 q = __ldg(p.overlay + (size_t)(obs0 + ag) * p.max_overlay + r);
            const int x0 = (int)(short)(q.x & 0xffff), y0 = (int)(short)(q.x >> 16);
            const int x1 = (int)(short)(q.y & 0xffff), y1 = (int)(short)(q.y >> 16);
            s_ov[ag * ov_slots + 2 * r] = make_int4(x0, y0, x1, y1);
            s_ov[ag * ov_slots + 2 * r + 1] = make_int4(q.z & 0xffffff, 0, 0, 0);
            const int cx0 = max(x0, 0), cy0 = max(y0, 0), cx1 = min(x1, W), cy1 = min(y1, H);
            if (cx0 < cx1 && cy0 < cy1)
                for (int ty = cy0 >> 2; ty <= ((cy1 - 1) >> 2); ++ty)
                    for (int tx = cx0 >> 3; tx <= ((cx1 - 1) >> 3); ++tx) {
                        const int t = ty * p.tiles_x + tx;
                        atomicOr(&s_ovtile[ag * ovt_words + (t >> 5)], 1u << (t & 31));
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
    mbar_wait_bounded(s_bar, 0, 8);       // completed phase: makes the staged bytes visible to this thread

    // ---- per-agent traversal set-up and box binning
    const int gx = p.gx, gz = p.gz;
    // voxel-index strides of the y-packed layout: x and z move by whole columns, y by single bits
    const int stride_x = 1 << p.lay.ysh, stride_z = gx << p.lay.ysh, stride_y = 1;
    // Traversal is confined to the cell box [lo, hi) that holds every filled voxel of this env
    // (nothing outside it can be hit), so rays that leave it, e.g. into the sky, stop there.
    const int lox = s_count[1], loy = s_count[2], loz = s_count[3];
    const int hix = s_count[4], hiy = s_count[5], hiz = s_count[6];
    const bool any_voxel = (lox < hix) && (loy < hiy) && (loz < hiz);
    const uint32_t vi_bias = OCC_SHARED ? 8u * smem_addr(smem) : 0u;
    const int P_ = p.palette;
    const uint32_t lut_base = smem_addr(s_lut);
    if (tid < kDdaVecs * apc) {
        // DDA start table of agent ag, entry 3*signs + axis (bit c of `signs` set: direction component c
        // negative): x = signed distance from the eye to the cell face the ray meets first, y = cells
        // left before the occupied box ends that way, z = voxel-index stride, w = shared-memory address
        // of the colour-table row of the face entered by a step along this axis.
        const int ag = tid / kDdaVecs, e = tid - ag * kDdaVecs;
        const int signs = e / 3, ax = e - 3 * signs, neg = (signs >> ax) & 1;
        const float4 c0 = s_agent[kAgentRecVecs * ag];
        const float Pc = ax == 0 ? c0.x : (ax == 1 ? c0.y : c0.z);
        const bool cam_in = any_voxel && (c0.x >= (float)lox) && (c0.x < (float)hix) && (c0.y >= (float)loy) &&
                            (c0.y < (float)hiy) && (c0.z >= (float)loz) && (c0.z < (float)hiz);
        int cx0 = 0, cy0 = 0, cz0 = 0;
        if (cam_in) { cx0 = (int)floorf(c0.x); cy0 = (int)floorf(c0.y); cz0 = (int)floorf(c0.z); }
        const int cc = ax == 0 ? cx0 : (ax == 1 ? cy0 : cz0);
        const int lo_c = ax == 0 ? lox : (ax == 1 ? loy : loz), hi_c = ax == 0 ? hix : (ax == 1 ? hiy : hiz);
        const int st = ax == 0 ? stride_x : (ax == 1 ? stride_y : stride_z);
        s_dda[kDdaVecs * ag + e] = make_float4(neg ? (float)cc - Pc : (float)(cc + 1) - Pc,
                                               neg ? (float)(cc - lo_c) : (float)(hi_c - 1 - cc),
                                               __int_as_float(neg ? -st : st),
                                               __uint_as_float(lut_base + (uint32_t)((2 * ax + neg) * P_ * 4)));
        if (e == 0) {
            const int vi0 = stride_x * cx0 + stride_z * cz0 + stride_y * cy0;
            const bool filled = cam_in && ((s_occ[vi0 >> 5] >> (vi0 & 31)) & 1u);
            float4 *slot = &s_agent[kAgentRecVecs * ag + 3];
            slot->x = __uint_as_float((uint32_t)vi0 + vi_bias);
            slot->y = __uint_as_float(__float_as_uint(slot->y) | (cam_in ? kAgentInside : 0u) | (filled ? 4u : 0u));
        }
    }
    {
        const int nb = min(s_count[0], p.max_boxes);
        for (int i = tid; i < apc * p.max_boxes; i += NT) {
            const int ag = i / p.max_boxes, b = i - ag * p.max_boxes;
            const float4 c0 = s_agent[kAgentRecVecs * ag], c1 = s_agent[kAgentRecVecs * ag + 1];
            const float4 c2 = s_agent[kAgentRecVecs * ag + 2];
            const float Px = c0.x, Py = c0.y, Pz = c0.z, Fx = c0.w, Fy = c1.x, Fz = c1.y;
            const float Rx = c1.z, Ry = c1.w, Rz = c2.x, Ux = c2.y, Uy = c2.z, Uz = c2.w;
            const int self_box = __float_as_int(s_agent[kAgentRecVecs * ag + 3].z);
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
            s_rel[2 * i] = make_float4(lx, ly, lz, front ? tmin * 0.9999f : 0.0f);
            s_rel[2 * i + 1] = make_float4(hx, hy, hz, B.z);
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
            uint32_t *mask = s_mask + (size_t)ag * ntiles * mw;
            for (int ty = py0 >> 2; ty <= (py1 >> 2); ++ty)
                for (int tx = px0 >> 3; tx <= (px1 >> 3); ++tx)
                    atomicOr(&mask[(ty * p.tiles_x + tx) * mw + (b >> 5)], bit);
        }
    }
    __syncthreads();

    const uint8_t *mat_env = p.mat + (size_t)env * ((size_t)gx * gz << p.lay.ysh) - vi_bias;
    const float flox = (float)lox, floy = (float)loy, floz = (float)loz;
    const float fhix = (float)hix, fhiy = (float)hiy, fhiz = (float)hiz;

    // ---- per-lane constants of the 8 x 4 tile: pixel offsets and the store plan.  Depth goes to the
    // lane's own pixel; lanes 0..23 each write one 32-bit word (row r, word j) of the tile's four
    // 24-byte RGB row segments, picked by a byte permute from the packed colours of pixels q0 and
    // q0+1 of that row.  keep() pins each of them in a register: recomputing them per tile costs
    // more issue slots than the registers are worth.
    constexpr int kWarps = NT / 32;
    float lane_a = (float)(2 * (lane & 7)), lane_b = (float)(2 * (lane >> 3));
    const int st_r = lane / 6, st_j = lane - 6 * st_r;
    const int st_q0 = (4 * st_j) / 3, st_byte = 4 * st_j - 3 * st_q0;       // first byte within pixel q0
    uint32_t st_src = (uint32_t)((st_r & 3) * 8 + st_q0);
    // bytes st_byte.. of pixel q0 (3 of them at most), then pixel q0+1 from its byte 0 (selector 4..)
    uint32_t st_sel = st_byte == 0 ? 0x4210u : (st_byte == 1 ? 0x5421u : 0x6542u);
    if (lane >= 24) st_sel = 0xffffffffu;                                   // marks the lanes that store no RGB word
    const int depth_lane_off = (lane >> 3) * W + (lane & 7);
    const int rgb_lane_off = st_r * W * 3 + st_j * 4;
    keep(lane_a); keep(lane_b); keep(st_src); keep(st_sel);
    const uint32_t tile_begin = smem_addr(s_tile) + 16u * (uint32_t)warp;
    const uint32_t tile_end = smem_addr(s_tile) + 16u * (uint32_t)ntiles;
    const uint32_t inside_row = lut_base + (uint32_t)(kFaceInside * P_ * 4);

    for (int ag = 0; ag < apc; ++ag) {
        const int obs = obs0 + ag;
        uint8_t *rgb_obs = p.rgb + (size_t)obs * H * W * 3;
        float *depth_obs = p.depth + (size_t)obs * H * W;
        const float4 c0 = s_agent[kAgentRecVecs * ag], c1 = s_agent[kAgentRecVecs * ag + 1];
        const float4 c2 = s_agent[kAgentRecVecs * ag + 2], c3 = s_agent[kAgentRecVecs * ag + 3];
        const uint32_t aflags = __float_as_uint(c3.y);
        if (aflags & kAgentBad) {                   // non-finite camera: a sky frame
            for (int i = tid; i < W * H; i += NT) depth_obs[i] = p.miss_depth;
            for (int i = tid; i < W * H * 3; i += NT) rgb_obs[i] = (uint8_t)(p.sky_rgbx >> (8 * (i % 3)));
            continue;
        }
        const float Px = c0.x, Py = c0.y, Pz = c0.z;
        const bool cam_in = (aflags & kAgentInside) != 0;
        uint32_t vi0 = __float_as_uint(c3.x);
        const uint32_t row0 = (aflags & 4u) ? inside_row : kNoRow;
        // exit-time factor: pulls the exit in by the rounding drift of the accumulated crossing times;
        // -inf (so that the product is -inf or NaN and the first test ends the walk) when the eye sits
        // in a filled voxel
        float escale = (aflags & 4u) ? -kInf : p.exit_scale;
        const int ov_count = __float_as_int(c3.w);
        uint32_t dda_base = smem_addr(s_dda + kDdaVecs * ag);
        uint32_t mask_p = smem_addr(s_mask + ((size_t)ag * ntiles + warp) * mw);
        const float4 *rel = s_rel + (size_t)ag * 2 * p.max_boxes;
        const int4 *ov = s_ov + ag * ov_slots;
        const uint32_t *ovtile = s_ovtile + ag * ovt_words;
        float *depth_lane = depth_obs + depth_lane_off;
        uint8_t *rgb_lane = rgb_obs + rgb_lane_off;
        keep(vi0); keep(escale); keep64(depth_lane); keep64(rgb_lane);
        const uint8_t *mat_lane = mat_env;
        const uint32_t cam_p = smem_addr(s_agent + kAgentRecVecs * ag);

        // ---- tiles: warp w takes tiles w, w + nwarps, ... (8 x 4 pixels, one per lane)
        for (uint32_t tile_p = tile_begin; tile_p < tile_end; tile_p += 16u * kWarps, mask_p += 4u * kWarps * (uint32_t)mw) {
            float Ta, Tb;
            int tile_px;
            uint32_t tile_no;
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=f"(Ta), "=f"(Tb), "=r"(tile_px), "=r"(tile_no) : "r"(tile_p));
            // ---- ray through the pixel centre: d = F + a*Rs + b*Us, a = 2px+1-W, b = H-1-2py
            // (the basis is re-read from shared memory per tile: three broadcast loads cost less than
            // nine registers held across the walk)
            float Fx, Fy, Fz, Rx, Ry, Rz, Ux, Uy, Uz, unused;
            asm volatile("ld.shared.f32 %0, [%1+12];" : "=f"(Fx) : "r"(cam_p));
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4+16];" : "=f"(Fy), "=f"(Fz), "=f"(Rx), "=f"(Ry) : "r"(cam_p));
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4+32];" : "=f"(Rz), "=f"(Ux), "=f"(Uy), "=f"(Uz) : "r"(cam_p));
            (void)unused;
            const float a = Ta + lane_a, bb = Tb - lane_b;
            float dx = fmaf(bb, Ux, fmaf(a, Rx, Fx));
            float dy = fmaf(bb, Uy, fmaf(a, Ry, Fy));
            float dz = fmaf(bb, Uz, fmaf(a, Rz, Fz));
            // a component that is exactly zero never crosses a cell face; 1e-30 keeps it that way
            // without infinities in the slab arithmetic
            dx = dx == 0.0f ? 1e-30f : dx;
            dy = dy == 0.0f ? 1e-30f : dy;
            dz = dz == 0.0f ? 1e-30f : dz;
            const float ix = fast_rcp(dx), iy = fast_rcp(dy), iz = fast_rcp(dz);
            const float dtx = fabsf(ix), dty = fabsf(iy), dtz = fabsf(iz);
            const uint32_t sgn3 = (__float_as_uint(dx) >> 31) | ((__float_as_uint(dy) >> 30) & 2u) |
                                  ((__float_as_uint(dz) >> 29) & 4u);      // bit c set: component c negative
            const uint32_t tab = dda_base + 48u * sgn3;
            // rows of the DDA table for this ray's signs: {distance to the first face, cells left, index
            // stride, colour-table row} per axis; the colour-table rows are fetched only where needed
            float qxx, qxy, qyx, qyy, qzx, qzy;
            int sx, sy, sz;
            {
                uint32_t u0, u1, u2;
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=f"(qxx), "=f"(qxy), "=r"(sx), "=r"(u0) : "r"(tab));
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4+16];" : "=f"(qyx), "=f"(qyy), "=r"(sy), "=r"(u1) : "r"(tab));
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4+32];" : "=f"(qzx), "=f"(qzy), "=r"(sz), "=r"(u2) : "r"(tab));
            }
            auto face_row = [&](int axis) {            // colour-table row of the face entered along `axis`
                uint32_t r;
                asm volatile("ld.shared.u32 %0, [%1+12];" : "=r"(r) : "r"(tab + 16u * (uint32_t)axis));
                return r;
            };

            // ---- start of the walk: cell, first crossing times, time at which the ray leaves the box
            float t0x, t0y, t0z, t_exit, t_hit = 0.0f;
            uint32_t vi = vi0, row = row0;
            if (cam_in) {
                t0x = qxx * ix;
                t0y = qyx * iy;
                t0z = qzx * iz;
                t_exit = min3f(fmaf(qxy, dtx, t0x), fmaf(qyy, dty, t0y), fmaf(qzy, dtz, t0z)) * escale;
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
                const int v = stride_x * cx + stride_z * cz + stride_y * cy;
                vi = (uint32_t)v + vi_bias;
                t0x = ((float)(cx + (ngx ? 0 : 1)) - Px) * ix;
                t0y = ((float)(cy + (ngy ? 0 : 1)) - Py) * iy;
                t0z = ((float)(cz + (ngz ? 0 : 1)) - Pz) * iz;
                t_exit = min3f(fmaf(ngx ? (float)(cx - lox) : (float)(hix - 1 - cx), dtx, t0x),
                               fmaf(ngy ? (float)(cy - loy) : (float)(hiy - 1 - cy), dty, t0y),
                               fmaf(ngz ? (float)(cz - loz) : (float)(hiz - 1 - cz), dtz, t0z)) * p.exit_scale;
                const bool filled = alive && ((s_occ[v >> 5] >> (v & 31)) & 1u);
                // entered through the box face of axis eaxis, or the eye is inside a solid
                if (filled) row = eaxis < 0 ? inside_row : face_row(eaxis);
                if (!alive || filled) t_exit = -kInf;
            }
#if MV_PROBE >= 1 && MV_PROBE < 9
            t_exit = -kInf;
#endif
            // The crossing times accumulate (t += dt), so after n steps they differ from the exact
            // products by up to n roundings; the exit time was pulled in by that bound, which keeps
            // the walk inside the box.
            // 3D-DDA written in PTX so that each step is a fixed short sequence of predicated
            // instructions (see MV_DDA_ADVANCE); four steps per trip of the bounded loop.
            {
                const int budget = p.max_steps;
                if constexpr (OCC_SHARED) {
                    asm volatile(MV_DDA_BODY
                                 : "+r"(vi), "+f"(t_hit), "+r"(row), "+f"(t0x), "+f"(t0y), "+f"(t0z)
                                 : "f"(dtx), "f"(dty), "f"(dtz), "r"(sx), "r"(sy), "r"(sz), "f"(t_exit), "r"(budget),
                                   "r"(tab), "l"(0ull)
                                 : "memory");
                } else {
                    asm volatile(MV_DDA_BODY_GLOBAL
                                 : "+r"(vi), "+f"(t_hit), "+r"(row), "+f"(t0x), "+f"(t0y), "+f"(t0z)
                                 : "f"(dtx), "f"(dty), "f"(dtz), "r"(sx), "r"(sy), "r"(sz), "f"(t_exit), "r"(budget),
                                   "r"(tab), "l"(s_occ)
                                 : "memory");
                }
            }
            __syncwarp();
            const bool vhit = row != kNoRow;

            // ---- voxel colour: one material byte from global memory, then the shaded table
            uint32_t rgbx = p.sky_rgbx;
            float depth = p.miss_depth;
            if (vhit) {
                const uint32_t m = __ldg(mat_lane + vi);
                asm("ld.shared.u32 %0, [%1];" : "=r"(rgbx) : "r"(row + 4u * m));
                depth = t_hit;
            }
#if MV_PROBE == 9
            depth = t_hit;
#endif

            // ---- boxes of this tile (skip those wholly behind every lane's voxel hit); a box wins
            // only with a strictly smaller time
            {
                uint32_t m;
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(m) : "r"(mask_p));
#if MV_PROBE >= 2 && MV_PROBE < 9
                m = 0;
#endif
                float tb = vhit ? t_hit : kInf;
                const float wmax = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(tb)));
                if (m != 0u || mw > 1) {
                    // signed reciprocals again: the index strides carry the signs of the direction
                    const float ix = __uint_as_float(__float_as_uint(dtx) | ((uint32_t)sx & 0x80000000u));
                    const float iy = __uint_as_float(__float_as_uint(dty) | ((uint32_t)sy & 0x80000000u));
                    const float iz = __uint_as_float(__float_as_uint(dtz) | ((uint32_t)sz & 0x80000000u));
                    uint32_t baddr = 0;
                    for (int w = 0;;) {
                        while (m) {
                            const int b = (__ffs(m) - 1) + 32 * w;
                            m &= m - 1;
                            const float4 lo = rel[2 * b], hi = rel[2 * b + 1];
                            if (lo.w > wmax) continue;
                            const float x1 = lo.x * ix, x2 = hi.x * ix, y1 = lo.y * iy, y2 = hi.y * iy;
                            const float z1 = lo.z * iz, z2 = hi.z * iz;
                            const float nx = fminf(x1, x2), ny = fminf(y1, y2), nz = fminf(z1, z2);
                            const float tn = max3f(nx, ny, nz);
                            const float tf = min3f(fmaxf(x1, x2), fmaxf(y1, y2), fmaxf(z1, z2));
                            const float t = fmaxf(tn, 0.0f);
                            if ((tn <= tf) && (tf > 0.0f) && (t < tb)) {
                                tb = t;
                                const uint32_t r = (tn < 0.0f) ? inside_row : face_row((nx == tn) ? 0 : ((ny == tn) ? 1 : 2));
                                baddr = r + 4u * __float_as_uint(hi.w);
                            }
                        }
                        if (++w >= mw) break;
                        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(m) : "r"(mask_p + 4u * (uint32_t)w));
                    }
                    if (baddr) {
                        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(rgbx) : "r"(baddr));
                        depth = tb + 0.0f;
                    }
                }
            }

            // ---- GUI overlay: rectangles in list order, later ones on top; depth is left alone
            if (ov_count > 0 && ((ovtile[tile_no >> 5] >> (tile_no & 31)) & 1u)) {
                const int px = (tile_px % W) + (lane & 7), py = (tile_px / W) + (lane >> 3);
                for (int r = 0; r < ov_count; ++r) {
                    const int4 q = ov[2 * r];
                    if (px >= q.x && px < q.z && py >= q.y && py < q.w) rgbx = (uint32_t)ov[2 * r + 1].x;
                }
            }

            // ---- store: depth rows are 32-byte segments; RGB rows are 24 bytes = 6 packed words
            depth_lane[tile_px] = depth;
            {
                const uint32_t ca = __shfl_sync(0xffffffffu, rgbx, st_src);
                const uint32_t cb = __shfl_sync(0xffffffffu, rgbx, st_src + 1);
                const uint32_t word = __byte_perm(ca, cb, st_sel);
                if ((int)st_sel >= 0) *reinterpret_cast<uint32_t *>(rgb_lane + 3 * tile_px) = word;
            }
        }
    }
}

}  // namespace mv
