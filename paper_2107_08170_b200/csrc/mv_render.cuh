// The render kernel: ray generation, grid traversal, box tests, shading and frame store for
// every observation of the batch in one launch (paper Section 3.2, Eq. 2).
//
// One CTA renders one observation.  A single bulk asynchronous copy stages the environment's
// block (1-bit occupancy grid, shaded colour table, box list) into shared memory; while it is
// in flight the CTA clears its per-tile box masks.  Boxes are then binned to 8x4-pixel screen
// tiles by the bounding rectangle of their projected corners (conservative, so every box that
// a pixel's ray can touch is tested for that pixel).  Tiles are dealt to warps round-robin;
// each lane owns one pixel of the tile: it walks the occupancy grid with a branch-free 3D-DDA
// in shared memory, tests the tile's candidate boxes with slab tests, looks the colour up in
// the shaded table and the warp writes 24-byte RGB row segments as packed 32-bit words and
// 32-byte depth row segments.
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

// Reciprocal to 1 ulp in one instruction; every use is inside toleranced intersection arithmetic.
__device__ __forceinline__ float fast_rcp(float x) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// One DDA step (see the loop in render_kernel): operands %3..%5 = dt, %6..%8 = t0, %9..%11 =
// index strides, %12 = grid-exit time, %14 = last occupancy word, %15 = shared base address
// (or %17 = 64-bit global base address when the occupancy does not fit shared memory).
#define MV_DDA_MOVE                                  \
    " min.f32 t, tx, ty, tz;\n"                      \
    " setp.geu.f32 pq, t, %12;\n"                    \
    " @pq bra MV_DDA_DONE;\n"                        \
    " setp.eq.f32 px, tx, t;\n"                      \
    " setp.eq.and.f32 py, ty, t, !px;\n"             \
    " or.pred pxy, px, py;\n"                        \
    " @px add.f32 kx, kx, 0f3F800000;\n"             \
    " @px add.s32 vi, vi, %9;\n"                    \
    " @py add.f32 ky, ky, 0f3F800000;\n"             \
    " @py add.s32 vi, vi, %10;\n"                    \
    " @!pxy add.f32 kz, kz, 0f3F800000;\n"           \
    " @!pxy add.s32 vi, vi, %11;\n"                  \
    " fma.rn.f32 tx, kx, %3, %6;\n"                  \
    " fma.rn.f32 ty, ky, %4, %7;\n"                 \
    " fma.rn.f32 tz, kz, %5, %8;\n"                 \
    " shr.u32 a, vi, 5;\n"                           \
    " min.u32 a, a, %14;\n"
#define MV_DDA_TEST                                  \
    " shf.r.wrap.b32 w, w, 0, vi;\n"                 \
    " and.b32 w, w, 1;\n"                            \
    " setp.ne.u32 pq, w, 0;\n"                       \
    " @pq bra MV_DDA_HIT;\n"
#define MV_DDA_STEP MV_DDA_MOVE " shl.b32 a, a, 2;\n add.u32 a, a, %15;\n ld.shared.u32 w, [a];\n" MV_DDA_TEST
#define MV_DDA_STEP_GLOBAL MV_DDA_MOVE " mad.wide.u32 ag, a, 4, %17;\n ld.global.nc.u32 w, [ag];\n" MV_DDA_TEST
#define MV_DDA_PROLOGUE                              \
    "{\n"                                            \
    " .reg .pred px, py, pxy, pq;\n"                 \
    " .reg .f32 t, tx, ty, tz, kx, ky, kz, th;\n"    \
    " .reg .u32 w, a, hit;\n"                        \
    " .reg .u64 ag;\n"                               \
    " .reg .s32 vi, it;\n"                           \
    " mov.f32 tx, %6;\n"                             \
    " mov.f32 ty, %7;\n"                            \
    " mov.f32 tz, %8;\n"                            \
    " mov.f32 kx, 0f00000000;\n"                     \
    " mov.f32 ky, 0f00000000;\n"                     \
    " mov.f32 kz, 0f00000000;\n"                     \
    " mov.f32 th, 0f00000000;\n"                     \
    " mov.u32 hit, 0;\n"                             \
    " mov.s32 vi, %16;\n"                            \
    " mov.s32 it, %13;\n"                            \
    "MV_DDA_LOOP:\n"
#define MV_DDA_EPILOGUE                              \
    " sub.u32 it, it, 2;\n"                          \
    " setp.gt.s32 pq, it, 0;\n"                      \
    " @pq bra MV_DDA_LOOP;\n"                        \
    " bra MV_DDA_DONE;\n"                            \
    "MV_DDA_HIT:\n"                                  \
    " mov.f32 th, t;\n"                              \
    " selp.u32 hit, 2, 3, py;\n"                     \
    " selp.u32 hit, 1, hit, px;\n"                   \
    "MV_DDA_DONE:\n"                                 \
    " mov.s32 %0, vi;\n"                             \
    " mov.f32 %1, th;\n"                             \
    " mov.u32 %2, hit;\n"                            \
    "}\n"

#ifndef MV_MINB
#define MV_MINB 3
#endif
// OCC_SHARED: the occupancy bits are staged in shared memory with the rest of the env block (the
// normal case); otherwise only the block's tail (colour table, boxes, bounds) is staged and the
// occupancy is read from global memory through the read-only path.
template <int NT, bool OCC_SHARED>
__global__ void __launch_bounds__(NT, MV_MINB) render_kernel(const RenderParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31;
    const int obs = p.obs_begin + blockIdx.x;
    const int env = obs / p.agents;
    const int W = p.W, H = p.H;

    // bytes of the env block that are NOT staged (the occupancy, when it stays in global memory)
    const uint32_t unstaged = OCC_SHARED ? 0u : p.lay.occ_bytes;
    const unsigned char *env_block = p.env_blocks + (size_t)env * p.lay.stride;
    const uint32_t *s_occ = OCC_SHARED ? reinterpret_cast<const uint32_t *>(smem)
                                       : reinterpret_cast<const uint32_t *>(env_block);
    const uint32_t *s_lut = reinterpret_cast<const uint32_t *>(smem + (p.lay.lut_off - unstaged));
    const float4 *s_box = reinterpret_cast<const float4 *>(smem + (p.lay.box_off - unstaged));
    const int *s_count = reinterpret_cast<const int *>(smem + (p.lay.count_off - unstaged));
    uint32_t *s_mask = reinterpret_cast<uint32_t *>(smem + p.smem_mask_off);
    float4 *s_rel = reinterpret_cast<float4 *>(smem + p.smem_rel_off);
    uint64_t *s_bar = reinterpret_cast<uint64_t *>(smem + p.smem_misc_off);
    int4 *s_ov = reinterpret_cast<int4 *>(smem + p.smem_ov_off);
    float4 *s_dda = reinterpret_cast<float4 *>(smem + p.smem_misc_off + 16);

    // ---- camera record (64 bytes, same for the whole CTA)
    const float4 *cq = reinterpret_cast<const float4 *>(p.cams + obs);
    const float4 c0 = __ldg(cq), c1 = __ldg(cq + 1), c2 = __ldg(cq + 2), c3 = __ldg(cq + 3);
    const float Px = c0.x, Py = c0.y, Pz = c0.z;
    const float Fx = c0.w, Fy = c1.x, Fz = c1.y;
    const float Rx = c1.z, Ry = c1.w, Rz = c2.x;
    const float Ux = c2.y, Uy = c2.z, Uz = c2.w;
    const int self_box = __float_as_int(c3.x);
    const uint32_t cam_flags = __float_as_uint(c3.y);

    uint8_t *rgb_obs = p.rgb + (size_t)obs * H * W * 3;
    float *depth_obs = p.depth + (size_t)obs * H * W;

    if (cam_flags & kFlagBadCamera) {          // non-finite camera: a sky frame, nothing staged
        for (int i = tid; i < W * H; i += NT) depth_obs[i] = p.miss_depth;
        for (int i = tid; i < W * H * 3; i += NT) rgb_obs[i] = (uint8_t)(p.sky_rgbx >> (8 * (i % 3)));
        return;
    }

    // ---- stage the environment block
    if (tid == 0) mbar_init(s_bar, 1);
    __syncthreads();
    if (tid == 0 && !p.skip_staging) {
        mbar_expect_tx(s_bar, p.lay.block_bytes - unstaged);
        bulk_load(smem, env_block + unstaged, p.lay.block_bytes - unstaged, s_bar);
    }
    const int ntiles = p.tiles_x * p.tiles_y;
    const int mw = p.mask_words;
    for (int i = tid; i < ntiles * mw; i += NT) s_mask[i] = 0u;
    // GUI rectangles of this observation (unpacked to x0,y0,x1,y1 / colour in two slots) and one
    // bit per tile that any rectangle touches, so untouched tiles pay a single bit test
    const int ov_count = p.overlay ? min(max(__ldg(p.overlay_count + obs), 0), p.max_overlay) : 0;
    uint32_t *s_ovtile = reinterpret_cast<uint32_t *>(s_ov + 2 * max(p.max_overlay, 1));
    if (ov_count > 0) {
        for (int i = tid; i < (ntiles + 31) / 32; i += NT) s_ovtile[i] = 0u;
        __syncthreads();
        if (tid < ov_count) {
            const int4 q = __ldg(p.overlay + (size_t)obs * p.max_overlay + tid);
            const int x0 = (int)(short)(q.x & 0xffff), y0 = (int)(short)(q.x >> 16);
            const int x1 = (int)(short)(q.y & 0xffff), y1 = (int)(short)(q.y >> 16);
            s_ov[2 * tid] = make_int4(x0, y0, x1, y1);
            s_ov[2 * tid + 1] = make_int4(q.z & 0xffffff, 0, 0, 0);
            const int cx0 = max(x0, 0), cy0 = max(y0, 0), cx1 = min(x1, W), cy1 = min(y1, H);
            if (cx0 < cx1 && cy0 < cy1)
                for (int ty = cy0 >> 2; ty <= ((cy1 - 1) >> 2); ++ty)
                    for (int tx = cx0 >> 3; tx <= ((cx1 - 1) >> 3); ++tx) {
                        const int t = ty * p.tiles_x + tx;
                        atomicOr(&s_ovtile[t >> 5], 1u << (t & 31));
                    }
        }
    }

    if (!mbar_wait_bounded(s_bar, 0, p.wait_polls)) {
        if (tid == 0) atomicOr(p.status, kFlagTimeout);
        mbar_wait_bounded(s_bar, 0, p.wait_polls);   // let a copy in flight land before leaving
        return;
    }
    __syncthreads();

    // ---- bin boxes to screen tiles
    const int gx = p.gx, gy = p.gy, gz = p.gz;
    {
        const float r2 = Rx * Rx + Ry * Ry + Rz * Rz, u2 = Ux * Ux + Uy * Uy + Uz * Uz;
        const float ir2 = 1.0f / r2, iu2 = 1.0f / u2;
        const int nb = min(s_count[0], p.max_boxes);
        for (int b = tid; b < p.max_boxes; b += NT) {
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
            s_rel[2 * b] = make_float4(lx, ly, lz, front ? tmin * 0.9999f : 0.0f);
            s_rel[2 * b + 1] = make_float4(hx, hy, hz, B.z);
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
            for (int ty = py0 >> 2; ty <= (py1 >> 2); ++ty)
                for (int tx = px0 >> 3; tx <= (px1 >> 3); ++tx)
                    atomicOr(&s_mask[(ty * p.tiles_x + tx) * mw + (b >> 5)], bit);
        }
    }
    __syncthreads();

    // ---- per-observation DDA set-up (uniform across the CTA)
    const int nvox = gx * gy * gz;
    const unsigned last_word = (unsigned)(nvox >> 5) - 1u;
    const int stride_z = gx, stride_y = gx * gz;
    // Traversal is confined to the cell box [lo, hi) that holds every filled voxel of this env
    // (nothing outside it can be hit), so rays that leave it, e.g. into the sky, stop there.
    const int lox = s_count[1], loy = s_count[2], loz = s_count[3];
    const int hix = s_count[4], hiy = s_count[5], hiz = s_count[6];
    const bool any_voxel = (lox < hix) && (loy < hiy) && (loz < hiz);
    const bool cam_in = any_voxel && (Px >= (float)lox) && (Px < (float)hix) && (Py >= (float)loy) &&
                        (Py < (float)hiy) && (Pz >= (float)loz) && (Pz < (float)hiz);
    int cx0 = 0, cy0 = 0, cz0 = 0;
    if (cam_in) { cx0 = (int)floorf(Px); cy0 = (int)floorf(Py); cz0 = (int)floorf(Pz); }
    const int vi0 = cx0 + stride_z * cz0 + stride_y * cy0;
    const bool start_filled = cam_in && ((s_occ[vi0 >> 5] >> (vi0 & 31)) & 1u);
    // DDA start table, entry 2*axis + (direction component negative): x = signed distance from the
    // eye to the cell face the ray meets first, y = cells left before the box ends that way,
    // z = voxel-index stride (as int bits).  Looked up per ray instead of recomputed.
    if (tid < 6) {
        const int ax = tid >> 1, neg = tid & 1;
        const int c0 = ax == 0 ? cx0 : (ax == 1 ? cy0 : cz0);
        const float Pc = ax == 0 ? Px : (ax == 1 ? Py : Pz);
        const int lo_c = ax == 0 ? lox : (ax == 1 ? loy : loz), hi_c = ax == 0 ? hix : (ax == 1 ? hiy : hiz);
        const int st = ax == 0 ? 1 : (ax == 1 ? stride_y : stride_z);
        s_dda[tid] = make_float4(neg ? (float)c0 - Pc : (float)(c0 + 1) - Pc,
                                 neg ? (float)(c0 - lo_c) : (float)(hi_c - 1 - c0),
                                 __int_as_float(neg ? -st : st), 0.0f);
    }
    __syncthreads();
    const int max_steps = gx + gy + gz + 3;
    const uint8_t *mat_env = p.mat + (size_t)env * nvox;
    const int P_ = p.palette;

    // ---- tiles: warp w takes tiles w, w + nwarps, ... (8 x 4 pixels, one per lane)
    constexpr int kWarps = NT / 32;
    const int warp = tid >> 5;
    int tyi = warp / p.tiles_x, txi = warp - tyi * p.tiles_x;
    const float lane_a = (float)(2 * (lane & 7)), lane_b = (float)(2 * (lane >> 3));
    // store plan, fixed per lane: depth goes to the lane's own pixel; lanes 0..23 each write one
    // 32-bit word (row r, word j) of the tile's four 24-byte RGB row segments, assembled from the
    // packed colours of pixels q0 and q0+1 of that row
    const int st_r = lane / 6, st_j = lane - 6 * st_r;
    const int st_q0 = (4 * st_j) / 3, st_shift = 8 * (4 * st_j - 3 * st_q0);
    const int st_src = (st_r & 3) * 8 + st_q0;
    const int depth_lane_off = (lane >> 3) * W + (lane & 7);
    const int rgb_lane_off = st_r * W * 3 + st_j * 4;
    int tile_px = (tyi * 4) * W + txi * 8;          // first pixel of the warp's current tile
    // a = 2px+1-W and b = H-1-2py of the lane's pixel, kept as floats (small integers: exact)
    float a = (float)(16 * txi + 1 - W) + lane_a, bb = (float)(H - 1 - 8 * tyi) - lane_b;
    for (int tile = warp; tile < ntiles; tile += kWarps) {
        // ---- ray through the pixel centre: d = F + a*Rs + b*Us, a = 2px+1-W, b = H-1-2py
        float dx = fmaf(bb, Ux, fmaf(a, Rx, Fx));
        float dy = fmaf(bb, Uy, fmaf(a, Ry, Fy));
        float dz = fmaf(bb, Uz, fmaf(a, Rz, Fz));
        // a component that is exactly zero never crosses a cell face; 1e-30 keeps it that way
        // without infinities in the slab arithmetic
        dx = dx == 0.0f ? 1e-30f : dx;
        dy = dy == 0.0f ? 1e-30f : dy;
        dz = dz == 0.0f ? 1e-30f : dz;
        const float ix = fast_rcp(dx), iy = fast_rcp(dy), iz = fast_rcp(dz);
        const bool ngx = dx < 0.0f, ngy = dy < 0.0f, ngz = dz < 0.0f;
        const float dtx = fabsf(ix), dty = fabsf(iy), dtz = fabsf(iz);
        const uint32_t bx_ = __float_as_uint(dx) >> 31, by_ = __float_as_uint(dy) >> 31, bz_ = __float_as_uint(dz) >> 31;
        const uint32_t sgn3 = bx_ | (by_ << 1) | (bz_ << 2);        // bit c set: component c negative
        const float4 qx = s_dda[0 + bx_];
        const float4 qy = s_dda[2 + by_];
        const float4 qz = s_dda[4 + bz_];
        const int sx = __float_as_int(qx.z), sy = __float_as_int(qy.z), sz = __float_as_int(qz.z);

        // ---- grid traversal: crossing times are t0 + k*dt with integer-valued k, so the exit
        // time below is bit-identical to the crossing that would leave the grid
        float t0x, t0y, t0z, t_exit, t_hit = 0.0f;
        int vi = vi0, axis0 = -1;
        bool vhit = start_filled;
        if (cam_in) {
            t0x = qx.x * ix;
            t0y = qy.x * iy;
            t0z = qz.x * iz;
            t_exit = fminf(fmaf(qx.y, dtx, t0x), fminf(fmaf(qy.y, dty, t0y), fmaf(qz.y, dtz, t0z)));
        } else {
            // eye outside the occupied box: clip the ray to it, start in the entry cell
            const float x1 = ((float)lox - Px) * ix, x2 = ((float)hix - Px) * ix;
            const float y1 = ((float)loy - Py) * iy, y2 = ((float)hiy - Py) * iy;
            const float z1 = ((float)loz - Pz) * iz, z2 = ((float)hiz - Pz) * iz;
            const float nrx = fminf(x1, x2), nry = fminf(y1, y2), nrz = fminf(z1, z2);
            const float tn = fmaxf(nrx, fmaxf(nry, nrz));
            const float tf = fminf(fmaxf(x1, x2), fminf(fmaxf(y1, y2), fmaxf(z1, z2)));
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
            vi = cx + stride_z * cz + stride_y * cy;
            axis0 = eaxis;
            t0x = ((float)(cx + (ngx ? 0 : 1)) - Px) * ix;
            t0y = ((float)(cy + (ngy ? 0 : 1)) - Py) * iy;
            t0z = ((float)(cz + (ngz ? 0 : 1)) - Pz) * iz;
            t_exit = fminf(fmaf(ngx ? (float)(cx - lox) : (float)(hix - 1 - cx), dtx, t0x),
                           fminf(fmaf(ngy ? (float)(cy - loy) : (float)(hiy - 1 - cy), dty, t0y),
                                 fmaf(ngz ? (float)(cz - loz) : (float)(hiz - 1 - cz), dtz, t0z)));
            vhit = alive && ((s_occ[vi >> 5] >> (vi & 31)) & 1u);
            if (!alive) t_exit = -kInf;
        }
        int loop_axis = 0;
        if (!vhit) {
            // 3D-DDA written in PTX so that each step is a fixed short sequence of predicated
            // instructions: t = min(tx,ty,tz); stop when t >= t_exit; step the axis whose crossing
            // time equals t (ties: x, then y, then z): k += 1, voxel index += stride, crossing time
            // = fma(k, dt, t0); test the voxel's occupancy bit.  Two steps per trip of the bounded
            // loop.  The word-index clamp never binds (the exit test keeps the index inside the
            // grid); it only guards the shared load.
            // All loop state lives in registers declared inside the block and the outputs are
            // written only after the last read of an input, so no operand can alias another.
            uint32_t hit;
            int vout;
            float th;
            if constexpr (OCC_SHARED) {
                asm volatile(MV_DDA_PROLOGUE MV_DDA_STEP MV_DDA_STEP MV_DDA_EPILOGUE
                             : "=r"(vout), "=f"(th), "=r"(hit)
                             : "f"(dtx), "f"(dty), "f"(dtz), "f"(t0x), "f"(t0y), "f"(t0z), "r"(sx), "r"(sy), "r"(sz),
                               "f"(t_exit), "r"((uint32_t)max_steps), "r"(last_word), "r"(smem_addr(smem)), "r"(vi)
                             : "memory");
            } else {
                asm volatile(MV_DDA_PROLOGUE MV_DDA_STEP_GLOBAL MV_DDA_STEP_GLOBAL MV_DDA_EPILOGUE
                             : "=r"(vout), "=f"(th), "=r"(hit)
                             : "f"(dtx), "f"(dty), "f"(dtz), "f"(t0x), "f"(t0y), "f"(t0z), "r"(sx), "r"(sy), "r"(sz),
                               "f"(t_exit), "r"((uint32_t)max_steps), "r"(last_word), "r"(0u), "r"(vi), "l"(s_occ)
                             : "memory");
            }
            vi = vout;
            if (hit) t_hit = th;
            vhit = hit != 0;
            loop_axis = (int)hit;
        }
        __syncwarp();
        // entered face: the axis of the last step (the loop reports 1 + axis at a hit), else the
        // box-entry axis, else none = eye inside a solid
        const int axis = loop_axis > 0 ? loop_axis - 1 : axis0;

        // ---- boxes of this tile (skip those wholly behind every lane's voxel hit)
        float tb = kInf;
        int bface = 0;
        uint32_t bmat = 0;
        {
            const float wmax = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(vhit ? t_hit : kInf)));
            for (int w = 0; w < mw; ++w) {
                uint32_t m = s_mask[tile * mw + w];
                while (m) {
                    const int b = (__ffs(m) - 1) + 32 * w;
                    m &= m - 1;
                    const float4 lo = s_rel[2 * b], hi = s_rel[2 * b + 1];
                    if (lo.w > wmax) continue;
                    const float x1 = lo.x * ix, x2 = hi.x * ix, y1 = lo.y * iy, y2 = hi.y * iy;
                    const float z1 = lo.z * iz, z2 = hi.z * iz;
                    const float nx = fminf(x1, x2), ny = fminf(y1, y2), nz = fminf(z1, z2);
                    const float tn = fmaxf(nx, fmaxf(ny, nz));
                    const float tf = fminf(fmaxf(x1, x2), fminf(fmaxf(y1, y2), fmaxf(z1, z2)));
                    const float t = fmaxf(tn, 0.0f);
                    if ((tn <= tf) && (tf > 0.0f) && (t < tb)) {
                        tb = t;
                        bmat = __float_as_uint(hi.w);
                        const int ax = (nx == tn) ? 0 : ((ny == tn) ? 1 : 2);
                        bface = (tn < 0.0f) ? kFaceInside : 2 * ax + (int)((sgn3 >> ax) & 1u);
                    }
                }
            }
        }

        // ---- resolve nearest (voxels win ties), shade from the table
        uint32_t rgbx = p.sky_rgbx;
        float depth = p.miss_depth;
        if (tb < kInf && (!vhit || tb < t_hit)) {
            rgbx = s_lut[bface * P_ + (int)bmat];
            depth = tb + 0.0f;
        } else if (vhit) {
            const int m = __ldg(mat_env + vi);
            const int face = axis < 0 ? kFaceInside : 2 * axis + (int)((sgn3 >> axis) & 1u);
            rgbx = s_lut[face * P_ + m];
            depth = t_hit + 0.0f;
        }

        // ---- GUI overlay: rectangles in list order, later ones on top; depth is left alone
        if (ov_count > 0 && ((s_ovtile[tile >> 5] >> (tile & 31)) & 1u)) {
            const int px = txi * 8 + (lane & 7), py = tyi * 4 + (lane >> 3);
            for (int r = 0; r < ov_count; ++r) {
                const int4 q = s_ov[2 * r];
                if (px >= q.x && px < q.z && py >= q.y && py < q.w) rgbx = (uint32_t)s_ov[2 * r + 1].x;
            }
        }

        // ---- store: depth rows are 32-byte segments; RGB rows are 24 bytes = 6 packed words
        depth_obs[tile_px + depth_lane_off] = depth;
        {
            const uint32_t ca = __shfl_sync(0xffffffffu, rgbx, st_src);
            const uint32_t cb = __shfl_sync(0xffffffffu, rgbx, (st_src + 1) & 31);
            const uint32_t word = __funnelshift_r(ca | (cb << 24), cb >> 8, st_shift);
            if (lane < 24) *reinterpret_cast<uint32_t *>(rgb_obs + (tile_px * 3 + rgb_lane_off)) = word;
        }
        txi += kWarps;
        tile_px += 8 * kWarps;
        a += (float)(16 * kWarps);
        while (txi >= p.tiles_x) { txi -= p.tiles_x; ++tyi; tile_px += 3 * W; a -= (float)(2 * W); bb -= 8.0f; }
    }
}

}  // namespace mv
