/*
 * CPU oracle for the batched Render step (paper Section 3.2, Eq. 2: O = Render(S)).
 *
 * TEST INFRASTRUCTURE ONLY.  This file defines what a rendered observation is; it is slow on
 * purpose and is never part of the product path.  Only the tests, the smoke check and the
 * benchmark's cpu-baseline leg may build or call it.  It shares no code, header, table or
 * helper with the CUDA library.
 *
 * What it computes.  The paper's renderer is a depth-tested rasteriser (Section 3.2); for
 * opaque geometry sampled once per pixel centre that is the visible-surface function: the
 * nearest intersection of the pixel's ray with the scene.  The scene of one environment is
 * the state the paper lists in Section 3.2 (walls, objects, agent bodies, cameras) in the
 * discretised form of Section 3.1: a voxel grid of material ids plus axis-aligned boxes.  The
 * oracle is that definition written out: for every pixel it tests the ray against EVERY
 * filled voxel and EVERY box with a slab test in double precision and keeps the nearest.
 * No grid traversal, no culling, no tiling.  Pixels are independent, so they are spread
 * over OpenMP threads; nothing else is parallel.
 *
 * Conventions the paper leaves open (all fixed here, listed as readings in the design notes):
 *   - y is up; voxel (i,j,k) is the unit cube [i,i+1]x[j,j+1]x[k,k+1]; grid[j][k][i], i fastest.
 *   - yaw 0 looks along +z and grows toward +x; pitch > 0 looks up; row 0 is the image top.
 *   - one ray per pixel centre, not normalised, forward component 1, so the ray parameter t
 *     is planar depth (distance along the view axis).
 *   - the camera basis is evaluated in double and rounded to float; the pixel direction is
 *     then two chained float fused multiply-adds, so any implementation can trace bit-identical
 *     rays; every intersection is evaluated in double from those float rays.
 *   - shading: Lambert term from one directional light plus ambient, per face, rounded half up
 *     to uint8 (the paper only says "dynamic shading and simulated lighting", Section 3).
 *
 * Parity pins: tests/test_oracle_pins.py checks this file against closed forms (single wall,
 * floor depth, empty world, mirror symmetry, a hand-worked 4x4 image, ray marching, ...).
 * The constants of the default scene (field of view, light direction, sky colour, miss depth,
 * body proportions) come from the workload definition, not from the paper: parity unpinned
 * for those constants only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    float lo[3], hi[3];
    uint32_t material, pad;
} mvo_box;

typedef struct {
    int32_t gx, gy, gz;
    int32_t max_boxes;
    int32_t width, height;
    int32_t palette_size;
    double hfov;
    double light_dir[3];
    double ambient;
    uint8_t sky_rgb[3];
    uint8_t pad;
    float miss_depth;
} mvo_desc;

enum { FACE_INSIDE = 6 };          /* faces 0..5 = -x,+x,-y,+y,-z,+z (outward normal) */
enum { CLASS_NONE = -1, CLASS_VOXEL = 0, CLASS_BOX = 1 };

typedef struct { int i, j, k, material; } filled_voxel;

/* Camera basis in double, rounded to float: out = {P, F, Rs, Us} (12 floats). */
void mvo_camera_basis(const float pos[3], float yaw, float pitch, double hfov, int W, int H,
                      float out[12])
{
    double sy = sin((double)yaw), cy = cos((double)yaw);
    double sp = sin((double)pitch), cp = cos((double)pitch);
    double F[3] = { cp * sy, sp, cp * cy };
    double R[3] = { cy, 0.0, -sy };
    double U[3] = { -sp * sy, cp, -sp * cy };
    double tx = tan(hfov / 2.0);
    double ty = tx * (double)H / (double)W;
    for (int c = 0; c < 3; ++c) {
        out[c] = pos[c];
        out[3 + c] = (float)F[c];
        out[6 + c] = (float)(R[c] * (tx / (double)W));
        out[9 + c] = (float)(U[c] * (ty / (double)H));
    }
}

/* Face intensities: ambient + (1-ambient)*max(0, n.L) for the six axis normals, ambient inside. */
void mvo_face_intensity(const double light_dir[3], double ambient, double out[7])
{
    double n = sqrt(light_dir[0] * light_dir[0] + light_dir[1] * light_dir[1] +
                    light_dir[2] * light_dir[2]);
    for (int axis = 0; axis < 3; ++axis) {
        double l = light_dir[axis] / n;
        double neg = -l > 0.0 ? -l : 0.0;      /* face 2*axis   has normal -e_axis */
        double pos = l > 0.0 ? l : 0.0;        /* face 2*axis+1 has normal +e_axis */
        out[2 * axis] = ambient + (1.0 - ambient) * neg;
        out[2 * axis + 1] = ambient + (1.0 - ambient) * pos;
    }
    out[FACE_INSIDE] = ambient;
}

/* Shaded colour table lut[face][material][c] = floor(palette*I_face + 0.5). */
void mvo_shade_lut(const uint8_t *palette, int P, const double light_dir[3], double ambient,
                   uint8_t *lut)
{
    double I[7];
    mvo_face_intensity(light_dir, ambient, I);
    for (int f = 0; f < 7; ++f)
        for (int m = 0; m < P; ++m)
            for (int c = 0; c < 3; ++c) {
                double v = floor((double)palette[m * 3 + c] * I[f] + 0.5);
                lut[(f * P + m) * 3 + c] = (uint8_t)(v > 255.0 ? 255.0 : v);
            }
}

/* Ray/box slab test in double.  Returns 1 on a hit and sets *t_hit and *face. */
static int slab(const double P[3], const double d[3], const double lo[3], const double hi[3],
                double *t_hit, int *face)
{
    double tn = -INFINITY, tf = INFINITY;
    int axis_n = -1;
    for (int c = 0; c < 3; ++c) {
        if (d[c] == 0.0) {
            if (P[c] < lo[c] || P[c] > hi[c]) return 0;
            continue;
        }
        double t1 = (lo[c] - P[c]) / d[c];
        double t2 = (hi[c] - P[c]) / d[c];
        double nr = t1 < t2 ? t1 : t2;
        double fr = t1 < t2 ? t2 : t1;
        if (nr > tn) { tn = nr; axis_n = c; }      /* strict: lowest axis wins a tie */
        if (fr < tf) tf = fr;
    }
    if (!(tn <= tf) || !(tf > 0.0)) return 0;
    if (tn < 0.0 || axis_n < 0) { *t_hit = 0.0; *face = FACE_INSIDE; return 1; }
    *t_hit = tn + 0.0;                         /* -0.0 -> +0.0 */
    *face = 2 * axis_n + (d[axis_n] > 0.0 ? 0 : 1);
    return 1;
}

static int finite3(const float *v) { return isfinite(v[0]) && isfinite(v[1]) && isfinite(v[2]); }

/*
 * Render `n` pixels of one observation.  pxy[2*q], pxy[2*q+1] = column, row of pixel q;
 * oxy (may be NULL) = sub-pixel offsets of the sample point in pixel units.  With a zero
 * offset the direction is the float expression d = fmaf(b, Us, fmaf(a, Rs, F)); with a
 * non-zero offset (used only by the silhouette-edge rule of the parity tests) the same
 * expression is evaluated in double at the displaced sample point.
 * Outputs per pixel q: rgb[3q..], depth[q], id[3q..] = (class, index, face).
 * Returns the number of threads used, or a negative value on bad arguments.
 */
int mvo_render_pixels(const mvo_desc *D, const uint8_t *grid, const mvo_box *boxes, int box_count,
                      const uint8_t *palette, const float cam_pos[3], float yaw, float pitch,
                      int self_box, int n, const int32_t *pxy, const double *oxy,
                      uint8_t *rgb, float *depth, int32_t *id)
{
    if (!D || !palette || !cam_pos || !pxy || !rgb || !depth || n < 0) return -1;
    const int gx = D->gx, gy = D->gy, gz = D->gz, W = D->width, H = D->height, Pn = D->palette_size;
    if (box_count > D->max_boxes) box_count = D->max_boxes;
    if (box_count < 0) box_count = 0;

    int bad_cam = !finite3(cam_pos) || !isfinite(yaw) || !isfinite(pitch);

    /* every filled voxel of this environment, in index order i + gx*(k + gz*j) */
    size_t nvox = grid ? (size_t)gx * gy * gz : 0, nfill = 0;
    for (size_t v = 0; v < nvox; ++v) nfill += grid[v] != 0;
    filled_voxel *fv = (filled_voxel *)malloc((nfill ? nfill : 1) * sizeof(filled_voxel));
    if (!fv) return -2;
    nfill = 0;
    for (int j = 0; j < gy && grid; ++j)
        for (int k = 0; k < gz; ++k)
            for (int i = 0; i < gx; ++i) {
                int m = grid[((size_t)j * gz + k) * gx + i];
                if (m) {
                    if (m >= Pn) m = Pn - 1;
                    fv[nfill].i = i; fv[nfill].j = j; fv[nfill].k = k; fv[nfill].material = m;
                    ++nfill;
                }
            }

    uint8_t *lut = (uint8_t *)malloc((size_t)7 * Pn * 3);
    if (!lut) { free(fv); return -2; }
    mvo_shade_lut(palette, Pn, D->light_dir, D->ambient, lut);

    float basis[12];
    mvo_camera_basis(cam_pos, yaw, pitch, D->hfov, W, H, basis);
    const float *Pf = basis, *Ff = basis + 3, *Rs = basis + 6, *Us = basis + 9;
    const double P[3] = { Pf[0], Pf[1], Pf[2] };

    int threads = 1;
#ifdef _OPENMP
    threads = omp_get_max_threads();
#pragma omp parallel for schedule(dynamic, 16)
#endif
    for (int q = 0; q < n; ++q) {
        int px = pxy[2 * q], py = pxy[2 * q + 1];
        double d[3];
        if (!oxy || (oxy[2 * q] == 0.0 && oxy[2 * q + 1] == 0.0)) {
            float a = (float)(2 * px + 1 - W);
            float b = (float)(H - 1 - 2 * py);
            for (int c = 0; c < 3; ++c) d[c] = (double)fmaf(b, Us[c], fmaf(a, Rs[c], Ff[c]));
        } else {
            double a = 2.0 * ((double)px + oxy[2 * q]) + 1.0 - (double)W;
            double b = (double)H - 1.0 - 2.0 * ((double)py + oxy[2 * q + 1]);
            for (int c = 0; c < 3; ++c) d[c] = (double)Ff[c] + a * (double)Rs[c] + b * (double)Us[c];
        }

        double best_t = INFINITY;
        int best_class = CLASS_NONE, best_face = 0, best_mat = 0;
        long best_index = -1;

        for (size_t v = 0; v < nfill && !bad_cam; ++v) {
            double lo[3] = { fv[v].i, fv[v].j, fv[v].k };
            double hi[3] = { fv[v].i + 1.0, fv[v].j + 1.0, fv[v].k + 1.0 };
            double t; int f;
            if (slab(P, d, lo, hi, &t, &f) && t < best_t) {   /* index order => lowest index wins ties */
                best_t = t; best_class = CLASS_VOXEL; best_face = f; best_mat = fv[v].material;
                best_index = fv[v].i + (long)gx * (fv[v].k + (long)gz * fv[v].j);
            }
        }
        for (int b = 0; b < box_count && !bad_cam; ++b) {
            if (b == self_box) continue;
            const mvo_box *bx = &boxes[b];
            if (!(bx->lo[0] < bx->hi[0] && bx->lo[1] < bx->hi[1] && bx->lo[2] < bx->hi[2])) continue;
            double lo[3] = { bx->lo[0], bx->lo[1], bx->lo[2] };
            double hi[3] = { bx->hi[0], bx->hi[1], bx->hi[2] };
            double t; int f;
            if (slab(P, d, lo, hi, &t, &f) && t < best_t) {   /* strict: voxels and lower boxes win ties */
                best_t = t; best_class = CLASS_BOX; best_face = f; best_index = b;
                best_mat = (int)(bx->material < (uint32_t)Pn ? bx->material : (uint32_t)(Pn - 1));
            }
        }

        if (best_class == CLASS_NONE) {
            rgb[3 * q] = D->sky_rgb[0]; rgb[3 * q + 1] = D->sky_rgb[1]; rgb[3 * q + 2] = D->sky_rgb[2];
            depth[q] = D->miss_depth;
        } else {
            const uint8_t *col = &lut[(best_face * Pn + best_mat) * 3];
            rgb[3 * q] = col[0]; rgb[3 * q + 1] = col[1]; rgb[3 * q + 2] = col[2];
            depth[q] = (float)best_t;
        }
        if (id) { id[3 * q] = best_class; id[3 * q + 1] = (int32_t)best_index; id[3 * q + 2] = best_class == CLASS_NONE ? -1 : best_face; }
    }
    free(lut);
    free(fv);
    return threads;
}

/* All W*H pixels of one observation, row-major, pixel centres. */
int mvo_render_obs(const mvo_desc *D, const uint8_t *grid, const mvo_box *boxes, int box_count,
                   const uint8_t *palette, const float cam_pos[3], float yaw, float pitch,
                   int self_box, uint8_t *rgb, float *depth, int32_t *id)
{
    if (!D) return -1;
    int n = D->width * D->height;
    int32_t *pxy = (int32_t *)malloc((size_t)(n ? n : 1) * 2 * sizeof(int32_t));
    if (!pxy) return -2;
    for (int py = 0; py < D->height; ++py)
        for (int px = 0; px < D->width; ++px) {
            pxy[2 * (py * D->width + px)] = px;
            pxy[2 * (py * D->width + px) + 1] = py;
        }
    int r = mvo_render_pixels(D, grid, boxes, box_count, palette, cam_pos, yaw, pitch, self_box,
                              n, pxy, NULL, rgb, depth, id);
    free(pxy);
    return r;
}

/* ------------------------------------------------------------------------------------------
 * Pixel-space GUI overlay (paper Appendix A.2: geometric primitives drawn in the agent's field
 * of view, e.g. the time-left bar).  Reading: a short list of axis-aligned filled rectangles in
 * pixel coordinates, half-open [x0,x1) x [y0,y1), clipped to the image, painted over the RGB
 * frame in list order (later rectangles on top); the depth channel is not touched.
 * Record layout (16 bytes): int16 x0, y0, x1, y1; uint8 r, g, b, pad; uint32 pad. */
typedef struct { int16_t x0, y0, x1, y1; uint8_t rgb[3]; uint8_t pad0; uint32_t pad1; } mvo_rect;

void mvo_overlay(int W, int H, const mvo_rect *rects, int count, uint8_t *rgb)
{
    for (int r = 0; r < count; ++r)
        for (int y = 0; y < H; ++y)
            for (int x = 0; x < W; ++x)
                if (x >= rects[r].x0 && x < rects[r].x1 && y >= rects[r].y0 && y < rects[r].y1) {
                    rgb[(y * W + x) * 3] = rects[r].rgb[0];
                    rgb[(y * W + x) * 3 + 1] = rects[r].rgb[1];
                    rgb[(y * W + x) * 3 + 2] = rects[r].rgb[2];
                }
}

/* ------------------------------------------------------------------------------------------
 * Agent motion with collision against the voxel grid (paper Section 3.1: movement and collision
 * checking for agents are continuous; Section 3.2, Eq. 1: S' = Physics(S, A), here only the
 * agent-body part of it).  Reading, since the paper gives no formula:
 *   yaw' = yaw + dyaw; pitch' = clamp(pitch + dpitch, -max_pitch, max_pitch)      (float)
 *   step = forward*(sin yaw', 0, cos yaw') + strafe*(cos yaw', 0, -sin yaw')      (double)
 *   x_try = (float)(x + step.x), z_try = (float)(z + step.z)
 *   the body is the box [x-hw, x+hw] x [y-below, y+above] x [z-hw, z+hw] (float arithmetic);
 *   the x move is kept iff the body at (x_try, y, z) lies inside the grid and touches no filled
 *   voxel; then the z move is tried the same way from the accepted x (axis-separated sliding).
 *   Cells touched along an axis: floor(lo) .. floor(hi), both ends included.
 * cam = {x, y, z, yaw, pitch} in/out; move = {forward, strafe, dyaw, dpitch};
 * shape = {hw, below, above}.  Returns bit 0 = x move kept, bit 1 = z move kept. */
static int body_free(const uint8_t *grid, int gx, int gy, int gz, float x, float y, float z,
                     const float shape[3])
{
    float lo[3] = { x - shape[0], y - shape[1], z - shape[0] };
    float hi[3] = { x + shape[0], y + shape[2], z + shape[0] };
    int g[3] = { gx, gy, gz }, c0[3], c1[3];
    for (int c = 0; c < 3; ++c) {
        if (!(lo[c] >= 0.0f) || !(hi[c] < (float)g[c])) return 0;      /* also rejects NaN */
        c0[c] = (int)floorf(lo[c]);
        c1[c] = (int)floorf(hi[c]);
    }
    for (int j = c0[1]; j <= c1[1]; ++j)
        for (int k = c0[2]; k <= c1[2]; ++k)
            for (int i = c0[0]; i <= c1[0]; ++i)
                if (grid[((size_t)j * gz + k) * gx + i]) return 0;
    return 1;
}

int mvo_move_agent(const uint8_t *grid, int gx, int gy, int gz, float cam[5], const float move[4],
                   const float shape[3], float max_pitch)
{
    float yaw = cam[3] + move[2];
    float pitch = cam[4] + move[3];
    if (pitch > max_pitch) pitch = max_pitch;
    if (pitch < -max_pitch) pitch = -max_pitch;
    double sy = sin((double)yaw), cy = cos((double)yaw);
    double sxd = (double)move[0] * sy + (double)move[1] * cy;
    double szd = (double)move[0] * cy - (double)move[1] * sy;
    float x_try = (float)((double)cam[0] + sxd);
    float z_try = (float)((double)cam[2] + szd);
    int kept = 0;
    float x = cam[0], z = cam[2];
    if (body_free(grid, gx, gy, gz, x_try, cam[1], z, shape)) { x = x_try; kept |= 1; }
    if (body_free(grid, gx, gy, gz, x, cam[1], z_try, shape)) { z = z_try; kept |= 2; }
    cam[0] = x; cam[2] = z; cam[3] = yaw; cam[4] = pitch;
    return kept;
}

/* ------------------------------------------------------------------------------------------
 * Greedy merging of voxels into boxes (paper Section 3.3: adjacent voxels are merged into a small
 * number of enclosing parallelepipeds by a greedy O(n) pass at the start of an episode).  The
 * paper does not spell the pass out; the reading used here is the usual greedy sweep: visit
 * voxels in index order (x fastest, then z, then y); at the first filled voxel not yet covered,
 * grow a box along +x while the material is the same and the cells are uncovered, then along +z
 * while the whole x-run qualifies, then along +y while the whole x-z slab qualifies; emit it and
 * mark it covered.  Materials are compared after clamping to the palette.
 * boxes_out: [max_out] records {lo x,y,z, hi x,y,z as float, material, 0}; returns the number of
 * boxes the pass produces (only the first max_out are written). */
int mvo_merge_voxels(const uint8_t *grid, int gx, int gy, int gz, int palette_size, mvo_box *boxes_out,
                     int max_out)
{
    size_t n = (size_t)gx * gy * gz;
    uint8_t *mat = (uint8_t *)malloc(n ? n : 1), *cov = (uint8_t *)calloc(n ? n : 1, 1);
    if (!mat || !cov) { free(mat); free(cov); return -2; }
    for (size_t v = 0; v < n; ++v) mat[v] = grid[v] >= palette_size ? (uint8_t)(palette_size - 1) : grid[v];
#define CELL(i, j, k) (((size_t)(j) * gz + (k)) * gx + (i))
#define OPEN(i, j, k, m) (grid[CELL(i, j, k)] != 0 && !cov[CELL(i, j, k)] && mat[CELL(i, j, k)] == (m))
    int count = 0;
    for (int j = 0; j < gy; ++j)
        for (int k = 0; k < gz; ++k)
            for (int i = 0; i < gx; ++i) {
                if (grid[CELL(i, j, k)] == 0 || cov[CELL(i, j, k)]) continue;
                int m = mat[CELL(i, j, k)];
                int w = 1, d = 1, h = 1;
                while (i + w < gx && OPEN(i + w, j, k, m)) ++w;
                for (;;) {
                    if (k + d >= gz) break;
                    int ok = 1;
                    for (int a = 0; a < w && ok; ++a) ok = OPEN(i + a, j, k + d, m);
                    if (!ok) break;
                    ++d;
                }
                for (;;) {
                    if (j + h >= gy) break;
                    int ok = 1;
                    for (int b = 0; b < d && ok; ++b)
                        for (int a = 0; a < w && ok; ++a) ok = OPEN(i + a, j + h, k + b, m);
                    if (!ok) break;
                    ++h;
                }
                for (int c = 0; c < h; ++c)
                    for (int b = 0; b < d; ++b)
                        for (int a = 0; a < w; ++a) cov[CELL(i + a, j + c, k + b)] = 1;
                if (count < max_out) {
                    mvo_box *o = &boxes_out[count];
                    o->lo[0] = (float)i; o->lo[1] = (float)j; o->lo[2] = (float)k;
                    o->hi[0] = (float)(i + w); o->hi[1] = (float)(j + h); o->hi[2] = (float)(k + d);
                    o->material = (uint32_t)m; o->pad = 0;
                }
                ++count;
            }
#undef CELL
#undef OPEN
    free(mat); free(cov);
    return count;
}
