// World-store and camera kernels: everything that turns the caller's arrays into the
// device-resident layout the render kernel stages (paper Section 3.3: geometry is prepared
// once per episode; Section 3.2: objects and cameras are state that changes every step).
#pragma once
#include "mv_device.cuh"

namespace mv {

// Four 0/non-zero bytes of a word -> 4 bits.
__device__ __forceinline__ uint32_t nz_bits4(uint32_t v) {
    const uint32_t ones = __vcmpne4(v, 0u) & 0x01010101u;
    return (ones * 0x01020408u) >> 24;
}

// 4 x 4 byte transpose: in[i] holds byte c of column c at height i; out[c] the four heights of column c.
__device__ __forceinline__ void transpose4x4(const uint32_t in[4], uint32_t out[4]) {
    const uint32_t a = __byte_perm(in[0], in[1], 0x5140), b = __byte_perm(in[2], in[3], 0x5140);   // c0h0 c0h1 c1h0 c1h1 | ..h2 h3
    const uint32_t c = __byte_perm(in[0], in[1], 0x7362), d = __byte_perm(in[2], in[3], 0x7362);   // c2h0 c2h1 c3h0 c3h1 | ..h2 h3
    out[0] = __byte_perm(a, b, 0x5410); out[1] = __byte_perm(a, b, 0x7632);
    out[2] = __byte_perm(c, d, 0x5410); out[3] = __byte_perm(c, d, 0x7632);
}

// Destination env of the e-th env of an upload: a contiguous range, or an index list.
__device__ __forceinline__ size_t upload_env(const int32_t *__restrict__ env_index, int env_begin, size_t e) {
    return env_index ? (size_t)__ldg(env_index + e) : (size_t)env_begin + e;
}

// uint8 grid [env][y][z][x] -> occupancy bits packed along y inside the env block (see EnvLayout)
// plus a material copy by voxel index with ids clamped to the palette.  One thread packs 32
// heights of four neighbouring columns: 32 four-byte loads, four words and 128 material bytes out.
__global__ void pack_grid_kernel(const uint8_t *__restrict__ grid, unsigned char *__restrict__ env_blocks,
                                 uint8_t *__restrict__ mat, EnvLayout lay, int gx, int gy, int gz, int env_begin,
                                 const int32_t *__restrict__ env_index, int env_count, int palette, uint32_t *status)
{
    const int xg_n = gx / 4, col_words = 1 << (lay.ysh - 5);
    const size_t per_env = (size_t)xg_n * gz * col_words;
    const size_t gid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= per_env * (size_t)env_count) return;
    const size_t e = gid / per_env;
    size_t r = gid - e * per_env;
    const int wq = (int)(r / ((size_t)xg_n * gz));
    r -= (size_t)wq * xg_n * gz;
    const int z = (int)(r / xg_n), xg = (int)(r - (size_t)z * xg_n);
    const size_t nvox = (size_t)gx * gy * gz;
    const uint8_t *src = grid + e * nvox + (size_t)z * gx + 4 * xg;
    const uint32_t cap = (uint32_t)(palette - 1) * 0x01010101u;
    uint32_t bits[4] = {0, 0, 0, 0}, clamped = 0;
    const size_t env = upload_env(env_index, env_begin, e);
    const uint32_t u0 = voxel_index(lay.ysh, gx, 4 * xg, 32 * wq, z);
    uint8_t *mdst = mat + env * ((size_t)gx * gz << lay.ysh) + u0;
    uint32_t col[4][8];                                 // material bytes: column c, heights 4k..4k+3 in word k
#pragma unroll
    for (int h0 = 0; h0 < 32; h0 += 4) {
        uint32_t v[4], t[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int y = 32 * wq + h0 + i;
            const uint32_t orig = y < gy ? __ldg(reinterpret_cast<const uint32_t *>(src + (size_t)y * gz * gx)) : 0u;
            const uint32_t nz = __vcmpne4(orig, 0u);               // 0xff per filled byte, decided before clamping
#pragma unroll
            for (int c = 0; c < 4; ++c) bits[c] |= ((nz >> (8 * c)) & 1u) << (h0 + i);
            const uint32_t cl = __vminu4(orig, cap);
            clamped |= cl ^ orig;
            v[i] = cl;
        }
        transpose4x4(v, t);
#pragma unroll
        for (int c = 0; c < 4; ++c) col[c][h0 / 4] = t[c];
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {                       // 32 contiguous bytes per column: two 16-byte stores
        uint4 *dst = reinterpret_cast<uint4 *>(mdst + ((size_t)c << lay.ysh));
        dst[0] = make_uint4(col[c][0], col[c][1], col[c][2], col[c][3]);
        dst[1] = make_uint4(col[c][4], col[c][5], col[c][6], col[c][7]);
    }
    uint32_t *occ = reinterpret_cast<uint32_t *>(env_blocks + env * lay.stride);
#pragma unroll
    for (int c = 0; c < 4; ++c) occ[(u0 >> 5) + ((uint32_t)c << (lay.ysh - 5))] = bits[c];
    if (clamped) atomicOr(status, kFlagMaterial);
}

// Cell box [lo, hi) that contains every filled voxel of an env, from the packed occupancy bits.
// One CTA per env; written next to the box count.  An empty grid gives lo > hi.
__global__ void occupied_bounds_kernel(unsigned char *__restrict__ env_blocks, EnvLayout lay, int env_begin,
                                       const int32_t *__restrict__ env_index, int gx, int gy, int gz)
{
    unsigned char *blk = env_blocks + upload_env(env_index, env_begin, blockIdx.x) * lay.stride;
    const uint32_t *occ = reinterpret_cast<const uint32_t *>(blk);
    const int wsh = lay.ysh - 5;                   // log2 of the words per column
    const int nwords = (gx * gz) << wsh;
    int lo[3] = {gx, gy, gz}, hi[3] = {-1, -1, -1};
    for (int w = threadIdx.x; w < nwords; w += blockDim.x) {
        const uint32_t m = occ[w];
        if (!m) continue;
        const int col = w >> wsh, y0 = (w - (col << wsh)) * 32;
        const int x = col % gx, z = col / gx;
        lo[0] = min(lo[0], x); hi[0] = max(hi[0], x);
        lo[1] = min(lo[1], y0 + __ffs(m) - 1); hi[1] = max(hi[1], y0 + 31 - __clz(m));
        lo[2] = min(lo[2], z); hi[2] = max(hi[2], z);
    }
    __shared__ int s_lo[3], s_hi[3];
    if (threadIdx.x < 3) { s_lo[threadIdx.x] = 1 << 30; s_hi[threadIdx.x] = -1; }
    __syncthreads();
#pragma unroll
    for (int c = 0; c < 3; ++c) {
        const int l = __reduce_min_sync(0xffffffffu, lo[c]), h = __reduce_max_sync(0xffffffffu, hi[c]);
        if ((threadIdx.x & 31) == 0) { atomicMin(&s_lo[c], l); atomicMax(&s_hi[c], h); }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int *dst = reinterpret_cast<int *>(blk + lay.count_off);
        dst[1] = s_lo[0]; dst[2] = s_lo[1]; dst[3] = s_lo[2];
        dst[4] = s_hi[0] + 1; dst[5] = s_hi[1] + 1; dst[6] = s_hi[2] + 1;
        dst[7] = 0;
    }
}

// Shaded colour table per env: lut[face][m] = RGBX of floor(palette*I_face + 0.5), in double.
__global__ void build_lut_kernel(const uint8_t *__restrict__ palette, unsigned char *__restrict__ env_blocks,
                                 EnvLayout lay, int env_begin, const int32_t *__restrict__ env_index, int env_count, int P,
                                 double lx, double ly, double lz, double ambient)
{
    const int gid = blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= env_count * kFaces * P) return;
    const int e = gid / (kFaces * P), r = gid - e * kFaces * P;
    const int f = r / P, m = r - f * P;
    double I = ambient;
    if (f < 6) {
        const double n = sqrt(__dadd_rn(__dadd_rn(__dmul_rn(lx, lx), __dmul_rn(ly, ly)), __dmul_rn(lz, lz)));
        const double comp = (f >> 1) == 0 ? lx : ((f >> 1) == 1 ? ly : lz);
        double l = comp / n;
        if (!(f & 1)) l = -l;                       // even faces have the negative normal
        l = l > 0.0 ? l : 0.0;
        I = __dadd_rn(ambient, __dmul_rn(__dsub_rn(1.0, ambient), l));
    }
    const uint8_t *pc = palette + ((size_t)e * P + m) * 3;
    uint32_t out = 0;
#pragma unroll
    for (int c = 0; c < 3; ++c) {
        double v = floor(__dadd_rn(__dmul_rn((double)pc[c], I), 0.5));
        v = v > 255.0 ? 255.0 : v;
        out |= (uint32_t)v << (8 * c);
    }
    uint32_t *lut = reinterpret_cast<uint32_t *>(env_blocks + upload_env(env_index, env_begin, e) * lay.stride + lay.lut_off);
    lut[f * P + m] = out;
}

// Box lists into the env blocks; material ids and counts are clamped.
__global__ void copy_boxes_kernel(const uint4 *__restrict__ boxes, const int32_t *__restrict__ counts,
                                  unsigned char *__restrict__ env_blocks, EnvLayout lay, int env_begin,
                                  const int32_t *__restrict__ env_index, int env_count, int max_boxes, int palette,
                                  uint32_t *status)
{
    const int gid = blockIdx.x * blockDim.x + threadIdx.x;
    const int per_env = max_boxes + 1;
    if (gid >= env_count * per_env) return;
    const int e = gid / per_env, b = gid - e * per_env;
    unsigned char *blk = env_blocks + upload_env(env_index, env_begin, e) * lay.stride;
    if (b == max_boxes) {
        int n = counts[e];
        if (n < 0 || n > max_boxes) { n = n < 0 ? 0 : max_boxes; atomicOr(status, kFlagBoxCount); }
        *reinterpret_cast<int *>(blk + lay.count_off) = n;
        return;
    }
    uint4 lo = boxes[((size_t)e * max_boxes + b) * 2], hi = boxes[((size_t)e * max_boxes + b) * 2 + 1];
    if (hi.z >= (uint32_t)palette) { hi.z = palette - 1; atomicOr(status, kFlagMaterial); }
    uint4 *dst = reinterpret_cast<uint4 *>(blk + lay.box_off) + 2 * b;
    dst[0] = lo;
    dst[1] = hi;
}

// Camera -> ray basis, evaluated in double and rounded to float:
// F = (cp*sy, sp, cp*cy), R = (cy, 0, -sy), U = (-sp*sy, cp, -sp*cy); Rs = R*kr, Us = U*ku
// with kr = tan(hfov/2)/W and ku = (tan(hfov/2)*H/W)/H computed on the host in double.
__device__ __forceinline__ void write_camrec(CamRec *out, float px, float py, float pz, float yaw, float pitch,
                                             int self_box, double kr, double ku, uint32_t *status)
{
    CamRec r;
    r.self_box = self_box;
    r.pad[0] = r.pad[1] = 0;
    const bool ok = isfinite(px) && isfinite(py) && isfinite(pz) && isfinite(yaw) && isfinite(pitch);
    r.flags = ok ? 0u : kFlagBadCamera;
    double sy, cy, sp, cp;
    sincos((double)(ok ? yaw : 0.0f), &sy, &cy);
    sincos((double)(ok ? pitch : 0.0f), &sp, &cp);
    r.P[0] = px; r.P[1] = py; r.P[2] = pz;
    r.F[0] = (float)__dmul_rn(cp, sy); r.F[1] = (float)sp; r.F[2] = (float)__dmul_rn(cp, cy);
    r.Rs[0] = (float)__dmul_rn(cy, kr); r.Rs[1] = (float)__dmul_rn(0.0, kr); r.Rs[2] = (float)__dmul_rn(-sy, kr);
    r.Us[0] = (float)__dmul_rn(__dmul_rn(-sp, sy), ku); r.Us[1] = (float)__dmul_rn(cp, ku);
    r.Us[2] = (float)__dmul_rn(__dmul_rn(-sp, cy), ku);
    *out = r;
    if (!ok) atomicOr(status, kFlagBadCamera);
}

__global__ void camera_kernel(const int32_t *__restrict__ cams, CamRec *__restrict__ out, int num_obs,
                              double kr, double ku, uint32_t *status)
{
    const int o = blockIdx.x * blockDim.x + threadIdx.x;
    if (o >= num_obs) return;
    const int32_t *c = cams + (size_t)o * 6;
    write_camrec(out + o, __int_as_float(c[0]), __int_as_float(c[1]), __int_as_float(c[2]),
                 __int_as_float(c[3]), __int_as_float(c[4]), c[5], kr, ku, status);
}

// True iff the body box around (x, y, z) lies inside the grid and touches no filled voxel
// (cells floor(lo)..floor(hi) on every axis, ends included).
__device__ __forceinline__ bool body_free(const uint32_t *occ, uint32_t ysh, int gx, int gy, int gz, float x, float y,
                                          float z, float hw, float below, float above)
{
    const float lx = __fsub_rn(x, hw), hx = __fadd_rn(x, hw);
    const float ly = __fsub_rn(y, below), hy = __fadd_rn(y, above);
    const float lz = __fsub_rn(z, hw), hz = __fadd_rn(z, hw);
    if (!(lx >= 0.0f) || !(hx < (float)gx) || !(ly >= 0.0f) || !(hy < (float)gy) || !(lz >= 0.0f) ||
        !(hz < (float)gz))
        return false;
    const int i0 = (int)floorf(lx), i1 = (int)floorf(hx), j0 = (int)floorf(ly), j1 = (int)floorf(hy);
    const int k0 = (int)floorf(lz), k1 = (int)floorf(hz);
    for (int j = j0; j <= j1; ++j)
        for (int k = k0; k <= k1; ++k)
            for (int i = i0; i <= i1; ++i) {
                const uint32_t v = voxel_index(ysh, gx, i, j, k);
                if ((occ[v >> 5] >> (v & 31)) & 1u) return false;
            }
    return true;
}

// Agent motion with voxel collision; one thread per agent.  Updates the caller's camera array,
// the ray-basis table and the agent's own body box inside its env block.
__global__ void move_agents_kernel(int32_t *__restrict__ cams, const float4 *__restrict__ moves,
                                   CamRec *__restrict__ recs, unsigned char *__restrict__ env_blocks,
                                   EnvLayout lay, int num_obs, int agents, int gx, int gy, int gz, int max_boxes,
                                   float hw, float below, float above, float max_pitch, double kr, double ku,
                                   uint32_t *status)
{
    const int o = blockIdx.x * blockDim.x + threadIdx.x;
    if (o >= num_obs) return;
    int32_t *c = cams + (size_t)o * 6;
    const float x = __int_as_float(c[0]), y = __int_as_float(c[1]), z = __int_as_float(c[2]);
    const float4 mv = moves[o];
    const float yaw = __fadd_rn(__int_as_float(c[3]), mv.z);
    float pitch = __fadd_rn(__int_as_float(c[4]), mv.w);
    pitch = pitch > max_pitch ? max_pitch : pitch;
    pitch = pitch < -max_pitch ? -max_pitch : pitch;
    double sy, cy;
    sincos((double)yaw, &sy, &cy);
    const double sxd = __dadd_rn(__dmul_rn((double)mv.x, sy), __dmul_rn((double)mv.y, cy));
    const double szd = __dsub_rn(__dmul_rn((double)mv.x, cy), __dmul_rn((double)mv.y, sy));
    const float x_try = (float)__dadd_rn((double)x, sxd);
    const float z_try = (float)__dadd_rn((double)z, szd);
    unsigned char *blk = env_blocks + (size_t)(o / agents) * lay.stride;
    const uint32_t *occ = reinterpret_cast<const uint32_t *>(blk);
    float nx = x, nz = z;
    if (body_free(occ, lay.ysh, gx, gy, gz, x_try, y, nz, hw, below, above)) nx = x_try;
    if (body_free(occ, lay.ysh, gx, gy, gz, nx, y, z_try, hw, below, above)) nz = z_try;
    c[0] = __float_as_int(nx); c[2] = __float_as_int(nz);
    c[3] = __float_as_int(yaw); c[4] = __float_as_int(pitch);
    const int self_box = c[5];
    write_camrec(recs + o, nx, y, nz, yaw, pitch, self_box, kr, ku, status);
    const int count = *reinterpret_cast<const int *>(blk + lay.count_off);
    if (self_box >= 0 && self_box < min(count, max_boxes)) {
        float *b = reinterpret_cast<float *>(blk + lay.box_off) + 8 * self_box;
        b[0] = __fsub_rn(nx, hw); b[1] = __fsub_rn(y, below); b[2] = __fsub_rn(nz, hw);
        b[3] = __fadd_rn(nx, hw); b[4] = __fadd_rn(y, above); b[5] = __fadd_rn(nz, hw);
    }
}

// Occupancy of the envs of one merge launch re-packed along x (bit v&31 of word v>>5, v = x + gx*(z + gz*y)),
// the order in which the merge sweeps.  One thread per output word; scratch, off the per-step path.
__global__ void xpack_kernel(const unsigned char *__restrict__ env_blocks, EnvLayout lay, int env_begin, int env_count,
                             int gx, int gy, int gz, uint32_t *__restrict__ out)
{
    const size_t nwords = (size_t)gx * gy * gz / 32;
    const size_t gid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= nwords * (size_t)env_count) return;
    const size_t e = gid / nwords, w = gid - e * nwords;
    const uint32_t *occ = reinterpret_cast<const uint32_t *>(env_blocks + (size_t)(env_begin + e) * lay.stride);
    uint32_t word = 0;
    for (int b = 0; b < 32; ++b) {
        const size_t v = w * 32 + b;
        const int x = (int)(v % gx), r = (int)(v / gx), z = r % gz, y = r / gz;
        const uint32_t u = voxel_index(lay.ysh, gx, x, y, z);
        word |= ((occ[u >> 5] >> (u & 31)) & 1u) << b;
    }
    out[gid] = word;
}

// Greedy merging of an env's voxels into boxes (paper Section 3.3), one warp per env, in the
// same order as a serial sweep: the warp finds the first filled, uncovered voxel in index order,
// grows a box along +x, then +z, then +y while every cell of the new row / slab is filled,
// uncovered and of the same material, emits it and marks it covered.  `occx` is the x-packed copy
// of the occupancy made by xpack_kernel; `covered` is scratch in the same packing, one bit per
// voxel per env of this launch, zeroed by the caller; it is read around L1 (ld.cg) because lanes
// read bits that other lanes set with atomics.
__global__ void merge_voxels_kernel(const uint32_t *__restrict__ occx, const uint8_t *__restrict__ mat,
                                    EnvLayout lay, int env_begin, int env_count, int gx, int gy, int gz,
                                    uint32_t *__restrict__ covered, uint4 *__restrict__ boxes_out,
                                    int32_t *__restrict__ count_out, int max_out)
{
    const int lane = threadIdx.x & 31;
    const int e = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (e >= env_count) return;
    const size_t nvox = (size_t)gx * gy * gz;
    const int nwords = (int)(nvox / 32);
    const uint32_t *occ = occx + (size_t)e * nwords;
    const uint8_t *m_env = mat + (size_t)(env_begin + e) * ((size_t)gx * gz << lay.ysh);
    uint32_t *cov = covered + (size_t)e * nwords;
    uint4 *out = boxes_out + (size_t)e * max_out * 2;
    const unsigned full = 0xffffffffu;
    auto open = [&](int i, int j, int k, int m) -> bool {
        const int v = i + gx * (k + gz * j);
        const uint32_t bit = 1u << (v & 31);
        return (occ[v >> 5] & bit) && !(__ldcg(&cov[v >> 5]) & bit) && m_env[voxel_index(lay.ysh, gx, i, j, k)] == m;
    };
    int count = 0;
    for (int w0 = 0; w0 < nwords; w0 += 32) {
        // words w0..w0+31: lane owns one; handle every uncovered filled voxel in them, in order
        // every trip covers at least one voxel of these 1024, so 1024 trips always suffice
        for (int trip = 0; trip < 1024; ++trip) {
            const int wi = w0 + lane;
            const uint32_t mine = wi < nwords ? (occ[wi] & ~__ldcg(&cov[wi])) : 0u;
            const unsigned has = __ballot_sync(full, mine != 0u);
            if (!has) break;
            const int src = __ffs(has) - 1;
            const uint32_t word = __shfl_sync(full, mine, src);
            const int v = (w0 + src) * 32 + (__ffs(word) - 1);
            const int i = v % gx, r = v / gx, k = r % gz, j = r / gz;
            const int m = m_env[voxel_index(lay.ysh, gx, i, j, k)];
            int w = 1, d = 1, h = 1;
            for (;;) {                                           // +x, 32 cells per vote
                const int a = w + lane;
                const bool ok = (i + a < gx) && open(i + a, j, k, m);
                const unsigned bad = ~__ballot_sync(full, ok);
                if (bad) { w += __ffs(bad) - 1; break; }
                w += 32;
            }
            for (; k + d < gz; ++d) {                            // +z, one row per trip
                bool ok = true;
                for (int a = lane; a < w; a += 32) ok = ok && open(i + a, j, k + d, m);
                if (!__all_sync(full, ok)) break;
            }
            for (; j + h < gy; ++h) {                            // +y, one slab per trip
                bool ok = true;
                for (int c = lane; c < w * d; c += 32) ok = ok && open(i + c % w, j + h, k + c / w, m);
                if (!__all_sync(full, ok)) break;
            }
            __syncwarp();
            // mark covered.  When gx is a multiple of 32, x-rows of different z or y never share a word:
            // one lane per row does plain read-modify-writes, and the warp barrier orders them before the
            // other lanes' later reads.  Narrower grids take atomics and a fence.
            if ((gx & 31) == 0) {
                for (int r = lane; r < d * h; r += 32) {
                    const int b = r % d, cc = r / d;
                    const int v0 = i + gx * ((k + b) + gz * (j + cc)), v1 = v0 + w;      // bits [v0, v1)
                    for (int wd = v0 >> 5; wd <= (v1 - 1) >> 5; ++wd) {
                        const int lo = max(v0 - 32 * wd, 0), hi = min(v1 - 32 * wd, 32);
                        const uint32_t bits = (hi == 32 ? 0xffffffffu : ((1u << hi) - 1u)) & ~((1u << lo) - 1u);
                        __stcg(&cov[wd], __ldcg(&cov[wd]) | bits);
                    }
                }
            } else {
                for (int c = lane; c < w * d * h; c += 32) {
                    const int a = c % w, b = (c / w) % d, cc = c / (w * d);
                    const int vv = (i + a) + gx * ((k + b) + gz * (j + cc));
                    atomicOr(&cov[vv >> 5], 1u << (vv & 31));
                }
                __threadfence();
            }
            __syncwarp();
            if (lane == 0 && count < max_out) {
                out[2 * count] = make_uint4(__float_as_uint((float)i), __float_as_uint((float)j),
                                            __float_as_uint((float)k), __float_as_uint((float)(i + w)));
                out[2 * count + 1] = make_uint4(__float_as_uint((float)(j + h)), __float_as_uint((float)(k + d)),
                                                (uint32_t)m, 0u);
            }
            ++count;
        }
    }
    if (lane == 0) count_out[e] = count;
}

// GUI rectangles into the library's table; counts clamped to 0..max_rects.
__global__ void copy_overlays_kernel(const int4 *__restrict__ rects, const int32_t *__restrict__ counts,
                                     int4 *__restrict__ out_rects, int32_t *__restrict__ out_counts, int num_obs,
                                     int max_rects)
{
    const int gid = blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= num_obs * (max_rects + 1)) return;
    const int o = gid / (max_rects + 1), r = gid - o * (max_rects + 1);
    if (r == max_rects) {
        const int n = rects ? counts[o] : 0;
        out_counts[o] = n < 0 ? 0 : (n > max_rects ? max_rects : n);
    } else if (rects) {
        out_rects[(size_t)o * max_rects + r] = rects[(size_t)o * max_rects + r];
    }
}

}  // namespace mv
