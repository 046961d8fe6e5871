// The render kernel: ray generation, grid traversal, box tests, shading and frame store for
// every observation of the batch in one launch (paper Section 3.2, Eq. 2).
//
// One CTA renders one observation.  A single bulk asynchronous copy stages the environment's
// block (1-bit occupancy grid, shaded colour table, box list) into shared memory; while it is
// in flight the CTA clears its per-tile box masks.  Boxes are then binned to 8x4-pixel screen
// tiles by the bounding rectangle of their projected corners (conservative, so every box that
// a pixel's ray can touch is tested for that pixel).  Warps pull tiles from a shared counter;
// each lane owns one pixel of the tile: it walks the occupancy grid with a 3D-DDA in shared
// memory, tests the tile's candidate boxes with slab tests, looks the colour up in the shaded
// table and the warp writes 24-byte RGB row segments as packed 32-bit words and 32-byte depth
// row segments.
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
constexpr int kWaitPolls = 1 << 18;

template <int NT>
__global__ void __launch_bounds__(NT, 3) render_kernel(const RenderParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31;
    const int obs = p.obs_begin + blockIdx.x;
    const int env = obs / p.agents;
    const int W = p.W, H = p.H;

    const uint32_t *s_occ = reinterpret_cast<const uint32_t *>(smem);
    const uint32_t *s_lut = reinterpret_cast<const uint32_t *>(smem + p.lay.lut_off);
    const float4 *s_box = reinterpret_cast<const float4 *>(smem + p.lay.box_off);
    const int *s_count = reinterpret_cast<const int *>(smem + p.lay.count_off);
    uint32_t *s_mask = reinterpret_cast<uint32_t *>(smem + p.smem_mask_off);
    float4 *s_rel = reinterpret_cast<float4 *>(smem + p.smem_rel_off);
    uint64_t *s_bar = reinterpret_cast<uint64_t *>(smem + p.smem_misc_off);
    int *s_next = reinterpret_cast<int *>(smem + p.smem_misc_off + 8);

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
    if (tid == 0) {
        mbar_init(s_bar, 1);
        *s_next = 0;
    }
    __syncthreads();
    if (tid == 0) {
        mbar_expect_tx(s_bar, p.lay.block_bytes);
        bulk_load(smem, p.env_blocks + (size_t)env * p.lay.stride, p.lay.block_bytes, s_bar);
    }
    const int ntiles = p.tiles_x * p.tiles_y;
    const int mw = p.mask_words;
    for (int i = tid; i < ntiles * mw; i += NT) s_mask[i] = 0u;

    if (!mbar_wait_bounded(s_bar, 0, kWaitPolls)) {
        if (tid == 0) atomicOr(p.status, kFlagTimeout);
        mbar_wait_bounded(s_bar, 0, kWaitPolls);   // let the copy in flight land before leaving
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
    const int stride_z = gx, stride_y = gx * gz;
    const bool cam_in = (Px >= 0.0f) && (Px < (float)gx) && (Py >= 0.0f) && (Py < (float)gy) &&
                        (Pz >= 0.0f) && (Pz < (float)gz);
    int cx0 = 0, cy0 = 0, cz0 = 0;
    if (cam_in) { cx0 = (int)floorf(Px); cy0 = (int)floorf(Py); cz0 = (int)floorf(Pz); }
    const int vi0 = cx0 + stride_z * cz0 + stride_y * cy0;
    const bool start_filled = cam_in && ((s_occ[vi0 >> 5] >> (vi0 & 31)) & 1u);
    const float fposx = (float)(cx0 + 1) - Px, fnegx = (float)cx0 - Px;
    const float fposy = (float)(cy0 + 1) - Py, fnegy = (float)cy0 - Py;
    const float fposz = (float)(cz0 + 1) - Pz, fnegz = (float)cz0 - Pz;
    const int max_steps = gx + gy + gz + 3;
    const uint8_t *mat_env = p.mat + (size_t)env * nvox;
    const int P_ = p.palette;

    for (;;) {
        int tile = 0;
        if (lane == 0) tile = atomicAdd(s_next, 1);
        tile = __shfl_sync(0xffffffffu, tile, 0);
        if (tile >= ntiles) break;
        const int tyi = tile / p.tiles_x, txi = tile - tyi * p.tiles_x;
        const int px = txi * 8 + (lane & 7), py = tyi * 4 + (lane >> 3);

        // ---- ray through the pixel centre (same fused expression as the definition)
        const float a = (float)(2 * px + 1 - W), bb = (float)(H - 1 - 2 * py);
        const float dx = fmaf(bb, Ux, fmaf(a, Rx, Fx));
        const float dy = fmaf(bb, Uy, fmaf(a, Ry, Fy));
        const float dz = fmaf(bb, Uz, fmaf(a, Rz, Fz));
        const float ix = 1.0f / dx, iy = 1.0f / dy, iz = 1.0f / dz;
        const bool parx = !(fabsf(ix) < kInf), pary = !(fabsf(iy) < kInf), parz = !(fabsf(iz) < kInf);
        const float dtx = parx ? 0.0f : fabsf(ix), dty = pary ? 0.0f : fabsf(iy), dtz = parz ? 0.0f : fabsf(iz);
        const int sx = dx >= 0.0f ? 1 : -1;
        const int sy = dy >= 0.0f ? stride_y : -stride_y;
        const int sz = dz >= 0.0f ? stride_z : -stride_z;

        // ---- grid traversal
        float t0x, t0y, t0z, t_exit, t_start = 0.0f;
        int vi = vi0, axis = -1;
        bool vhit = start_filled, alive = true;
        if (cam_in) {
            t0x = parx ? kInf : (dx >= 0.0f ? fposx : fnegx) * ix;
            t0y = pary ? kInf : (dy >= 0.0f ? fposy : fnegy) * iy;
            t0z = parz ? kInf : (dz >= 0.0f ? fposz : fnegz) * iz;
            const float nx = dx >= 0.0f ? (float)(gx - 1 - cx0) : (float)cx0;
            const float ny = dy >= 0.0f ? (float)(gy - 1 - cy0) : (float)cy0;
            const float nz = dz >= 0.0f ? (float)(gz - 1 - cz0) : (float)cz0;
            t_exit = fminf(fmaf(nx, dtx, t0x), fminf(fmaf(ny, dty, t0y), fmaf(nz, dtz, t0z)));
        } else {
            // eye outside the grid: clip the ray to the grid's box, start in the entry cell
            float tn = -kInf, tf = kInf;
            const float Pc[3] = {Px, Py, Pz}, ic[3] = {ix, iy, iz}, gc[3] = {(float)gx, (float)gy, (float)gz};
            const bool par[3] = {parx, pary, parz};
#pragma unroll
            for (int c = 0; c < 3; ++c) {
                if (par[c]) {
                    if (Pc[c] < 0.0f || Pc[c] > gc[c]) alive = false;
                } else {
                    const float t1 = (0.0f - Pc[c]) * ic[c], t2 = (gc[c] - Pc[c]) * ic[c];
                    const float nr = fminf(t1, t2), fr = fmaxf(t1, t2);
                    if (nr > tn) { tn = nr; axis = c; }
                    tf = fminf(tf, fr);
                }
            }
            if (!(tn <= tf) || !(tf > 0.0f)) alive = false;
            if (tn < 0.0f) axis = -1;
            t_start = fmaxf(tn, 0.0f);
            if (!alive) t_start = 0.0f;
            int cx = min(max((int)floorf(fmaf(t_start, dx, Px)), 0), gx - 1);
            int cy = min(max((int)floorf(fmaf(t_start, dy, Py)), 0), gy - 1);
            int cz = min(max((int)floorf(fmaf(t_start, dz, Pz)), 0), gz - 1);
            if (axis == 0) cx = dx > 0.0f ? 0 : gx - 1;
            if (axis == 1) cy = dy > 0.0f ? 0 : gy - 1;
            if (axis == 2) cz = dz > 0.0f ? 0 : gz - 1;
            vi = cx + stride_z * cz + stride_y * cy;
            t0x = parx ? kInf : ((float)(cx + (dx >= 0.0f ? 1 : 0)) - Px) * ix;
            t0y = pary ? kInf : ((float)(cy + (dy >= 0.0f ? 1 : 0)) - Py) * iy;
            t0z = parz ? kInf : ((float)(cz + (dz >= 0.0f ? 1 : 0)) - Pz) * iz;
            const float nx = dx >= 0.0f ? (float)(gx - 1 - cx) : (float)cx;
            const float ny = dy >= 0.0f ? (float)(gy - 1 - cy) : (float)cy;
            const float nz = dz >= 0.0f ? (float)(gz - 1 - cz) : (float)cz;
            t_exit = fminf(fmaf(nx, dtx, t0x), fminf(fmaf(ny, dty, t0y), fmaf(nz, dtz, t0z)));
            vhit = alive && ((s_occ[vi >> 5] >> (vi & 31)) & 1u);
            if (!alive) t_exit = -kInf;
        }
        float t_hit = t_start;
        if (!vhit) {
            float tx = t0x, ty = t0y, tz = t0z, kx = 0.0f, ky = 0.0f, kz = 0.0f;
#pragma unroll 1
            for (int it = 0; it < max_steps; ++it) {
                const float t = fminf(tx, fminf(ty, tz));
                if (!(t < t_exit)) break;
                if (tx == t)      { vi += sx; kx += 1.0f; tx = fmaf(kx, dtx, t0x); axis = 0; }
                else if (ty == t) { vi += sy; ky += 1.0f; ty = fmaf(ky, dty, t0y); axis = 1; }
                else              { vi += sz; kz += 1.0f; tz = fmaf(kz, dtz, t0z); axis = 2; }
                if ((unsigned)vi >= (unsigned)nvox) break;           // cannot happen; guards the read
                if ((s_occ[vi >> 5] >> (vi & 31)) & 1u) { vhit = true; t_hit = t; break; }
            }
        }
        __syncwarp();

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
                        const float ds = ax == 0 ? dx : (ax == 1 ? dy : dz);
                        bface = (tn < 0.0f) ? kFaceInside : 2 * ax + (ds > 0.0f ? 0 : 1);
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
            const float ds = axis == 0 ? dx : (axis == 1 ? dy : dz);
            const int face = axis < 0 ? kFaceInside : 2 * axis + (ds > 0.0f ? 0 : 1);
            rgbx = s_lut[face * P_ + m];
            depth = t_hit + 0.0f;
        }

        // ---- store: depth rows are 32-byte segments; RGB rows are 24 bytes = 6 packed words
        depth_obs[(size_t)py * W + px] = depth;
        {
            const int r = lane / 6, j = lane - 6 * r;          // lanes 0..23: row r, word j of the row
            const int q0 = (4 * j) / 3, o = 4 * j - 3 * q0;    // first pixel and byte offset in it
            const int src = (r & 3) * 8 + q0;
            const uint32_t ca = __shfl_sync(0xffffffffu, rgbx, src);
            const uint32_t cb = __shfl_sync(0xffffffffu, rgbx, (src + 1) & 31);
            const uint32_t lo = (ca & 0xffffffu) | (cb << 24), hi = (cb & 0xffffffu) >> 8;
            const uint32_t word = __funnelshift_r(lo, hi, 8 * o);
            if (lane < 24) {
                uint32_t *dst = reinterpret_cast<uint32_t *>(rgb_obs + ((size_t)(tyi * 4 + r) * W + txi * 8) * 3) + j;
                *dst = word;
            }
        }
    }
}

}  // namespace mv
