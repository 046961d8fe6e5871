// Host side of the C ABI declared in include/mv.h: argument checks, allocation of the
// device-resident world store, and the kernel launches.  No rendering arithmetic runs here.
#define MV_ENABLE_TEST_HOOKS
#include "../../include/mv.h"
#include "mv_device.cuh"
#include "mv_pack.cuh"
#include "mv_render.cuh"

#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

using namespace mv;

namespace {

#ifndef MV_NT
#define MV_NT 384
#endif
constexpr int kRenderThreads = MV_NT;          // threads per CTA of the render kernel...
constexpr int kRenderThreadsSmall = MV_NT / 2; // ...and for CTAs with few tiles (small images): twice as many, shorter CTAs per SM
// Below this many tiles per CTA the small shape is faster when there are CTAs enough to fill the GPU with it
// (measured: 64x36 images +10 %; 128x72 -2 %; four CTAs alone on the GPU -20 %: fewer warps per CTA, longer CTA).
constexpr int kSmallCtaTiles = 192;
constexpr int kHostChunks = 8;
// Staging + set-up of a CTA, in units of one observation's render time, as measured on B200 at 128x72:
// 0.15 to 0.18 for 64x16x64 grids, 0.10 for 128x32x128 grids (where a second agent's tables usually cost
// the third resident CTA per SM, which the occupancy query below sees).
constexpr double kCtaFixedCost = 0.15;
#ifndef MV_MERGE_SCRATCH_MB
#define MV_MERGE_SCRATCH_MB 1024
#endif
constexpr size_t kMergeScratchBytes = (size_t)MV_MERGE_SCRATCH_MB << 20;   // coverage bitmap for the envs of one merge launch

inline uint32_t round_up(uint32_t v, uint32_t a) { return (v + a - 1) / a * a; }

}  // namespace

struct mv_batch {
    mv_batch_desc desc;
    int num_obs = 0;
    size_t nvox = 0;
    size_t mat_bytes_per_env = 0;       // material store: one byte per voxel index (columns padded to 2^ysh)
    EnvLayout lay{};
    unsigned char *d_env_blocks = nullptr;
    uint8_t *d_mat = nullptr;
    CamRec *d_cams = nullptr;
    uint32_t *d_status = nullptr;
    uint32_t *d_covered = nullptr;      // merge scratch: one bit per voxel for merge_chunk envs
    int merge_chunk = 0;
    int4 *d_overlay = nullptr;          // [O][max_overlay_rects]
    int32_t *d_overlay_count = nullptr; // [O]
    int32_t *d_env_index = nullptr;     // [E] destination envs of a scattered upload (mv_upload_worlds_at)
    // host-side readiness tracking (per env)
    std::vector<uint8_t> has_grid, has_palette;
    int missing_grid = 0, missing_palette = 0;
    bool has_cams = false;
    double kr = 0, ku = 0;
    uint32_t sky_rgbx = 0;
    struct Smem { uint32_t tile_off, agent_off, agent_stride, agent_ov_off, agent_mask_off, agent_ovtile_off, misc_off, bytes; };
    Smem smem{};                        // shared-memory layout of the render kernel for agents_per_cta
    int agents_per_cta = 1;             // observations one CTA renders: 1, or every agent of its env
    int threads = MV_NT;                // threads per CTA of the render kernel (fewer for CTAs with few tiles)
    int sms = 0;
    int tiles_x = 0, tiles_y = 0, mask_words = 0;
    int64_t launches = 0;
    int wait_polls = 1 << 18;
    bool occ_shared = true;             // occupancy staged in shared memory (else read from global)
    bool occ_fits_shared = true;
    int smem_max = 0;                   // opt-in shared memory per CTA of the device
    int auto_agents_per_cta = 1;        // the library's own choice (a test hook can override it)
    int skip_staging = 0;
    int last_cuda_error = 0;
    // mv_step_host resources (allocated on first use)
    uint8_t *d_rgb = nullptr;
    float *d_depth = nullptr;
    mv_camera *d_cam_in = nullptr;
    mv_box *d_box_in = nullptr;
    int32_t *d_count_in = nullptr;
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_chunk[kHostChunks] = {};
    cudaEvent_t ev_done = nullptr;
    bool host_ready = false;
};

namespace {

int cuda_fail(mv_batch *b, cudaError_t e) {
    if (b) b->last_cuda_error = (int)e;
    return e == cudaErrorMemoryAllocation ? MV_ERR_OUT_OF_MEMORY : MV_ERR_CUDA;
}

#define MV_CUDA(b, call)                                   \
    do {                                                   \
        cudaError_t e_ = (call);                           \
        if (e_ != cudaSuccess) return cuda_fail((b), e_);  \
    } while (0)

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard() { if (ok && prev >= 0) cudaSetDevice(prev); }
};

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Shared-memory layout of the render kernel when one CTA renders `apc` observations of an env:
// staged env block, tile table, then one block per agent (camera record and DDA start table,
// eye-relative boxes, overlay rectangles, per-tile box masks, per-tile overlay bits), then the
// barrier and flag words.
mv_batch::Smem smem_layout(const mv_batch *b, int apc) {
    const mv_batch_desc &d = b->desc;
    const uint32_t ntiles = (uint32_t)(b->tiles_x * b->tiles_y);
    mv_batch::Smem m{};
    m.tile_off = round_up(b->lay.block_bytes, 16);
    m.agent_off = m.tile_off + ntiles * 16;
    m.agent_ov_off = kAgentRelOff + (uint32_t)(d.max_boxes > 0 ? d.max_boxes : 1) * 32;
    m.agent_mask_off = m.agent_ov_off + (uint32_t)(d.max_overlay_rects > 0 ? d.max_overlay_rects : 1) * 32;
    // per tile: the box-mask words, preceded by a summary word when there is more than one
    const uint32_t words_per_tile = b->mask_words > 1 ? (uint32_t)b->mask_words + 1 : 1u;
    m.agent_ovtile_off = m.agent_mask_off + round_up(ntiles * words_per_tile * 4, 16);
    m.agent_stride = m.agent_ovtile_off + round_up(((ntiles + 31) / 32) * 4, 16);
    m.misc_off = m.agent_off + (uint32_t)apc * m.agent_stride;
    m.bytes = m.misc_off + 32;
#if defined(MV_BRICKS) && MV_BRICKS == 1
    m.bytes += round_up((uint32_t)((d.grid_x / 4) * (d.grid_z / 4)), 16);   // experiment: one byte per column of 4x4x4 bricks
#endif
    return m;
}

// Threads per CTA: the small shape for CTAs with few tiles, if the batch has CTAs enough to fill the GPU
// six to an SM.
int pick_threads(const mv_batch *b, int apc) {
    const bool few_tiles = b->tiles_x * b->tiles_y * apc < kSmallCtaTiles;
    const bool fills = (int64_t)b->num_obs / apc >= (int64_t)6 * b->sms;
    return few_tiles && fills ? kRenderThreadsSmall : kRenderThreads;
}

// The three instantiations of the render kernel: column-word walk (grid at most 32 high, occupancy
// staged), indexed walk with staged occupancy, indexed walk with the occupancy in global memory.
using RenderFn = void (*)(const RenderParams);
RenderFn render_fn(const mv_batch *b) {
    if (b->threads == kRenderThreadsSmall) {
        if (!b->occ_shared) return render_kernel<kRenderThreadsSmall, false, false>;
        return b->lay.ysh == 5 ? render_kernel<kRenderThreadsSmall, true, true> : render_kernel<kRenderThreadsSmall, true, false>;
    }
    if (!b->occ_shared) return render_kernel<kRenderThreads, false, false>;
    return b->lay.ysh == 5 ? render_kernel<kRenderThreads, true, true> : render_kernel<kRenderThreads, true, false>;
}

int launch_render(mv_batch *b, uint8_t *d_rgb, float *d_depth, int obs_begin, int obs_count, cudaStream_t s) {
    RenderParams p{};
    p.env_blocks = b->d_env_blocks;
    p.mat = b->d_mat;
    p.cams = b->d_cams;
    p.rgb = d_rgb;
    p.depth = d_depth;
    p.status = b->d_status;
    p.lay = b->lay;
    p.obs_begin = obs_begin;
    p.obs_count = obs_count;
    p.agents = b->desc.agents_per_env;
    p.gx = b->desc.grid_x; p.gy = b->desc.grid_y; p.gz = b->desc.grid_z;
    p.max_boxes = b->desc.max_boxes;
    p.palette = b->desc.palette_size;
    p.W = b->desc.width; p.H = b->desc.height;
    p.tiles_x = b->tiles_x; p.tiles_y = b->tiles_y; p.mask_words = b->mask_words;
    p.sky_rgbx = b->sky_rgbx;
    p.miss_depth = b->desc.miss_depth;
    const uint32_t unstaged = b->occ_shared ? 0u : b->lay.occ_bytes;   // shared-memory offsets shift down by it
    p.smem_tile_off = b->smem.tile_off - unstaged; p.smem_agent_off = b->smem.agent_off - unstaged;
    p.smem_misc_off = b->smem.misc_off - unstaged;
    p.agent_stride = b->smem.agent_stride; p.agent_ov_off = b->smem.agent_ov_off;
    p.agent_mask_off = b->smem.agent_mask_off; p.agent_ovtile_off = b->smem.agent_ovtile_off;
    p.agents_per_cta = b->agents_per_cta;
    p.max_steps = b->desc.grid_x + b->desc.grid_y + b->desc.grid_z + 3;
    // accumulated crossing times drift from the exact products by at most one rounding per step
    p.exit_scale = 1.0f - (float)(b->desc.grid_x + b->desc.grid_y + b->desc.grid_z + 3) * 1.1920929e-7f;
    p.overlay = b->d_overlay;
    p.overlay_count = b->d_overlay_count;
    p.max_overlay = b->desc.max_overlay_rects;
    p.wait_polls = b->wait_polls;
    p.skip_staging = b->skip_staging;
    const int ctas = obs_count / b->agents_per_cta;   // callers pass whole environments when a CTA renders one
    render_fn(b)<<<ctas, b->threads, b->smem.bytes - unstaged, s>>>(p);
    b->launches++;
    MV_CUDA(b, cudaGetLastError());
    return MV_OK;
}

int launch_cameras(mv_batch *b, const mv_camera *d_cams, cudaStream_t s) {
    const int n = b->num_obs;
    camera_kernel<<<(n + 127) / 128, 128, 0, s>>>(reinterpret_cast<const int32_t *>(d_cams), b->d_cams, n,
                                                   b->kr, b->ku, b->d_status);
    b->launches++;
    MV_CUDA(b, cudaGetLastError());
    b->has_cams = true;
    return MV_OK;
}

int launch_boxes(mv_batch *b, int env_begin, const int32_t *d_env_index, int env_count, const mv_box *d_boxes,
                 const int32_t *d_count, cudaStream_t s) {
    const int n = env_count * (b->desc.max_boxes + 1);
    copy_boxes_kernel<<<(n + 255) / 256, 256, 0, s>>>(reinterpret_cast<const uint4 *>(d_boxes), d_count,
                                                       b->d_env_blocks, b->lay, env_begin, d_env_index, env_count,
                                                       b->desc.max_boxes, b->desc.palette_size, b->d_status);
    b->launches++;
    MV_CUDA(b, cudaGetLastError());
    return MV_OK;
}

// First-use resources of mv_step_host: all of them or none, so that a failed attempt can be retried.
void free_host_step(mv_batch *b) {
    cudaFree(b->d_rgb); cudaFree(b->d_depth); cudaFree(b->d_cam_in); cudaFree(b->d_box_in); cudaFree(b->d_count_in);
    b->d_rgb = nullptr; b->d_depth = nullptr; b->d_cam_in = nullptr; b->d_box_in = nullptr; b->d_count_in = nullptr;
    if (b->copy_stream) cudaStreamDestroy(b->copy_stream);
    b->copy_stream = nullptr;
    for (auto &ev : b->ev_chunk) { if (ev) cudaEventDestroy(ev); ev = nullptr; }
    if (b->ev_done) cudaEventDestroy(b->ev_done);
    b->ev_done = nullptr;
    b->host_ready = false;
}

int alloc_host_step(mv_batch *b) {
    const size_t px = (size_t)b->desc.width * b->desc.height;
    const size_t O = (size_t)b->num_obs, E = (size_t)b->desc.num_envs;
    cudaError_t e = cudaMalloc(&b->d_rgb, O * px * 3);
    if (e == cudaSuccess) e = cudaMalloc(&b->d_depth, O * px * 4);
    if (e == cudaSuccess) e = cudaMalloc(&b->d_cam_in, O * sizeof(mv_camera));
    if (e == cudaSuccess && b->desc.max_boxes > 0) {
        e = cudaMalloc(&b->d_box_in, E * b->desc.max_boxes * sizeof(mv_box));
        if (e == cudaSuccess) e = cudaMalloc(&b->d_count_in, E * sizeof(int32_t));
    }
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&b->copy_stream, cudaStreamNonBlocking);
    for (auto &ev : b->ev_chunk)
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&b->ev_done, cudaEventDisableTiming);
    if (e != cudaSuccess) {
        free_host_step(b);
        cudaGetLastError();
        return cuda_fail(b, e);
    }
    b->host_ready = true;
    return MV_OK;
}

// End of a synchronous host step: wait for the stream, then report a staging wait that ran out
// (the frames of such a step are not valid).
int finish_host_step(mv_batch *b, cudaStream_t s) {
    uint32_t word = 0;
    MV_CUDA(b, cudaMemcpyAsync(&word, b->d_status, 4, cudaMemcpyDeviceToHost, s));
    MV_CUDA(b, cudaStreamSynchronize(s));
    return (word & kFlagTimeout) ? MV_ERR_DEVICE_TIMEOUT : MV_OK;
}

}  // namespace

// ---- fixed scratch for mv_step_host_static -------------------------------------------------
// Lives in the library image: every GPU that loads the library holds these bytes until the
// process exits.  In host code the array's name is only a host-side stand-in, never a device
// address; the address a kernel or a copy may use comes from cudaGetSymbolAddress, taken once
// per device with that device current.
#define MV_STATIC_SCRATCH_BYTES (8u << 20)
static __device__ __align__(256) unsigned char g_static_scratch[MV_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
unsigned char *g_static_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on `device` (which must be current).  First use on a
// device asks the runtime for the symbol's address; later uses return the cached pointer.
int static_scratch_for_device(mv_batch *b, int device, unsigned char **out) {
    if (device < 0 || device >= kMaxDevices) return MV_ERR_UNSUPPORTED;
    if (!g_static_scratch_ptr[device]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) return cuda_fail(b, e);
        g_static_scratch_ptr[device] = static_cast<unsigned char *>(p);
    }
    *out = g_static_scratch_ptr[device];
    return MV_OK;
}
}  // namespace

namespace {
// Body of both upload entry points.  h_env_index: null for the contiguous range that starts at
// env_begin, else the (validated) destination env of each uploaded env.
int upload_worlds(mv_batch *b, int env_begin, const int32_t *h_env_index, int env_count, const uint8_t *d_grid,
                  const mv_box *d_boxes, const int32_t *d_box_count, const uint8_t *d_palette, cudaStream_t s) {
    if (d_boxes && !d_box_count) return MV_ERR_INVALID_ARG;
    if (d_boxes && b->desc.max_boxes == 0) return MV_ERR_INVALID_ARG;
    if ((d_grid && !aligned16(d_grid)) || (d_boxes && !aligned16(d_boxes))) return MV_ERR_INVALID_ARG;
    if (env_count == 0) return MV_OK;
    DeviceGuard g(b->desc.device);
    if (!g.ok) return MV_ERR_CUDA;
    const int32_t *d_index = nullptr;
    if (h_env_index) {
        // The list is copied in stream order into a buffer the batch owns; an earlier scattered upload
        // on another stream that has not finished would be overwritten (one stream at a time).
        MV_CUDA(b, cudaMemcpyAsync(b->d_env_index, h_env_index, (size_t)env_count * 4, cudaMemcpyHostToDevice, s));
        d_index = b->d_env_index;
    }
    auto dst_env = [&](int i) { return h_env_index ? h_env_index[i] : env_begin + i; };
    if (d_grid) {
        const size_t threads = ((size_t)(b->desc.grid_x / 4) * b->desc.grid_z << (b->lay.ysh - 5)) * (size_t)env_count;
        const size_t blocks = (threads + 255) / 256;
        if (blocks > 0x7fffffffull) return MV_ERR_INVALID_ARG;
        pack_grid_kernel<<<(unsigned)blocks, 256, 0, s>>>(d_grid, b->d_env_blocks, b->d_mat, b->lay, b->desc.grid_x,
                                                           b->desc.grid_y, b->desc.grid_z, env_begin, d_index, env_count,
                                                           b->desc.palette_size, b->d_status);
        b->launches++;
        MV_CUDA(b, cudaGetLastError());
        occupied_bounds_kernel<<<env_count, 256, 0, s>>>(b->d_env_blocks, b->lay, env_begin, d_index, b->desc.grid_x,
                                                          b->desc.grid_y, b->desc.grid_z);
        b->launches++;
        MV_CUDA(b, cudaGetLastError());
        for (int i = 0; i < env_count; ++i) {
            const int e = dst_env(i);
            if (!b->has_grid[e]) { b->has_grid[e] = 1; b->missing_grid--; }
        }
    }
    if (d_palette) {
        const int n = env_count * kFaces * b->desc.palette_size;
        build_lut_kernel<<<(n + 255) / 256, 256, 0, s>>>(d_palette, b->d_env_blocks, b->lay, env_begin, d_index, env_count,
                                                          b->desc.palette_size, (double)b->desc.light_dir[0],
                                                          (double)b->desc.light_dir[1], (double)b->desc.light_dir[2],
                                                          (double)b->desc.ambient);
        b->launches++;
        MV_CUDA(b, cudaGetLastError());
        for (int i = 0; i < env_count; ++i) {
            const int e = dst_env(i);
            if (!b->has_palette[e]) { b->has_palette[e] = 1; b->missing_palette--; }
        }
    }
    if (d_boxes) {
        int r = launch_boxes(b, env_begin, d_index, env_count, d_boxes, d_box_count, s);
        if (r != MV_OK) return r;
    }
    return MV_OK;
}
}  // namespace

extern "C" {

const char *mv_status_string(int status) {
    switch (status) {
        case MV_OK: return "ok";
        case MV_ERR_INVALID_ARG: return "invalid argument";
        case MV_ERR_OUT_OF_MEMORY: return "out of memory";
        case MV_ERR_CUDA: return "CUDA runtime error";
        case MV_ERR_NOT_READY: return "worlds or cameras not uploaded yet";
        case MV_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case MV_ERR_UNSUPPORTED: return "configuration exceeds a documented limit";
        default: return status > 0 ? "data-error flags set" : "unknown status";
    }
}

int mv_create_batch(const mv_batch_desc *desc, mv_batch **out) {
    if (!desc || !out) return MV_ERR_INVALID_ARG;
    *out = nullptr;
    const mv_batch_desc &d = *desc;
    auto dim_ok = [](int g) { return g >= 4 && g <= 1024 && (g % 4) == 0; };
    if (d.num_envs < 1 || d.agents_per_env < 1 || !dim_ok(d.grid_x) || !dim_ok(d.grid_y) || !dim_ok(d.grid_z) ||
        d.max_boxes < 0 || d.max_boxes > 256 || d.width < 8 || d.width > 4096 || (d.width % 8) != 0 ||
        d.height < 4 || d.height > 4096 || (d.height % 4) != 0 || d.palette_size < 1 || d.palette_size > 256 ||
        !(d.hfov_rad > 0.0f) || !(d.hfov_rad < 3.14159f) || !(d.ambient >= 0.0f) || !(d.ambient <= 1.0f) ||
        !std::isfinite(d.miss_depth) || d.device < 0 || d.max_overlay_rects < 0 || d.max_overlay_rects > 16)
        return MV_ERR_INVALID_ARG;
    const double ln = (double)d.light_dir[0] * d.light_dir[0] + (double)d.light_dir[1] * d.light_dir[1] +
                      (double)d.light_dir[2] * d.light_dir[2];
    if (!(ln > 0.0) || !std::isfinite(ln)) return MV_ERR_INVALID_ARG;
    if ((int64_t)d.num_envs * d.agents_per_env > (1 << 30)) return MV_ERR_INVALID_ARG;

    mv_batch *b = new (std::nothrow) mv_batch();
    if (!b) return MV_ERR_OUT_OF_MEMORY;
    b->desc = d;
    b->num_obs = d.num_envs * d.agents_per_env;
    b->nvox = (size_t)d.grid_x * d.grid_y * d.grid_z;
    b->has_grid.assign(d.num_envs, 0);
    b->has_palette.assign(d.num_envs, 0);
    b->missing_grid = b->missing_palette = d.num_envs;

    EnvLayout &L = b->lay;
    L.ysh = 5;                                              // bits per (x, z) column: a power of two >= grid_y, >= 32
    while ((1 << L.ysh) < d.grid_y) L.ysh++;
    L.occ_bytes = (uint32_t)(((size_t)d.grid_x * d.grid_z << L.ysh) / 8);
    b->mat_bytes_per_env = (size_t)d.grid_x * d.grid_z << L.ysh;
    L.lut_off = L.occ_bytes;
    L.box_off = L.lut_off + round_up(kFaces * d.palette_size * 4, 16);
    L.count_off = L.box_off + (uint32_t)d.max_boxes * 32;
    L.block_bytes = L.count_off + 32;
    L.stride = round_up(L.block_bytes, 128);

    b->tiles_x = d.width / 8;
    b->tiles_y = d.height / 4;
    b->mask_words = d.max_boxes > 0 ? (d.max_boxes + 31) / 32 : 1;
    b->smem = smem_layout(b, 1);

    // kr = tan(hfov/2)/W, ku = (tan(hfov/2)*H/W)/H in double (scalar set-up for the camera kernel)
    const double tx = std::tan((double)d.hfov_rad / 2.0);
    const double ty = tx * (double)d.height / (double)d.width;
    b->kr = tx / (double)d.width;
    b->ku = ty / (double)d.height;
    b->sky_rgbx = (uint32_t)d.sky_rgb[0] | ((uint32_t)d.sky_rgb[1] << 8) | ((uint32_t)d.sky_rgb[2] << 16);

    int ndev = 0;
    cudaError_t e = cudaGetDeviceCount(&ndev);
    if (e != cudaSuccess || d.device >= ndev) { delete b; return e != cudaSuccess ? MV_ERR_CUDA : MV_ERR_INVALID_ARG; }
    DeviceGuard g(d.device);
    if (!g.ok) { delete b; return MV_ERR_CUDA; }
    int smem_max = 0, sms = 0;
    e = cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, d.device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, d.device);
    if (e != cudaSuccess) { delete b; return MV_ERR_CUDA; }
    b->smem_max = smem_max;
    // the occupancy normally rides in shared memory with the rest of the env block; a grid too large
    // for that keeps it in global memory and stages only the block's tail
    b->occ_fits_shared = (int)b->smem.bytes <= smem_max;
    b->occ_shared = b->occ_fits_shared;
    if ((int)(b->smem.bytes - L.occ_bytes) > smem_max) { delete b; return MV_ERR_UNSUPPORTED; }
    // The dynamic shared-memory cap is a property of the kernel function on this device, shared by
    // every batch: raise it to the device's maximum once, never to one batch's own size.
    for (RenderFn f : {RenderFn(render_kernel<kRenderThreads, true, true>), RenderFn(render_kernel<kRenderThreads, true, false>),
                       RenderFn(render_kernel<kRenderThreads, false, false>), RenderFn(render_kernel<kRenderThreadsSmall, true, true>),
                       RenderFn(render_kernel<kRenderThreadsSmall, true, false>),
                       RenderFn(render_kernel<kRenderThreadsSmall, false, false>)})
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max);
    if (e != cudaSuccess) { delete b; return MV_ERR_CUDA; }
    // One CTA per environment (block staged once for all its agents) when that still fills the GPU;
    // otherwise one CTA per observation.  Cost model: waves of resident CTAs x (agents + fixed part).
    if (d.agents_per_env > 1) {
        const mv_batch::Smem all = smem_layout(b, d.agents_per_env);
        const uint32_t unstaged = b->occ_shared ? 0u : L.occ_bytes;   // never give up staged occupancy for it
        if ((int)(all.bytes - unstaged) <= smem_max) {
            auto waves_cost = [&](const mv_batch::Smem &m, int apc) {
                int per_sm = 0;
                cudaError_t q = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, render_fn(b), kRenderThreads,
                                                                              m.bytes - unstaged);
                if (q != cudaSuccess || per_sm < 1) return 1e30;
                const double slots = (double)per_sm * sms, ctas = (double)b->num_obs / apc;
                return std::ceil(ctas / slots) * (apc + kCtaFixedCost);
            };
            if (waves_cost(all, d.agents_per_env) < waves_cost(b->smem, 1)) {
                b->smem = all;
                b->agents_per_cta = b->auto_agents_per_cta = d.agents_per_env;
            }
        }
    }

    b->sms = sms;
    b->threads = pick_threads(b, b->agents_per_cta);

    const size_t blocks_bytes = (size_t)d.num_envs * L.stride;
    bool ok = cudaMalloc(&b->d_env_blocks, blocks_bytes) == cudaSuccess &&
              cudaMalloc(&b->d_mat, (size_t)d.num_envs * b->mat_bytes_per_env) == cudaSuccess &&
              cudaMalloc(&b->d_cams, (size_t)b->num_obs * sizeof(CamRec)) == cudaSuccess &&
              cudaMalloc(&b->d_status, 16) == cudaSuccess &&
              cudaMalloc(&b->d_env_index, (size_t)d.num_envs * 4) == cudaSuccess;
    if (ok && d.max_overlay_rects > 0)
        ok = cudaMalloc(&b->d_overlay, (size_t)b->num_obs * d.max_overlay_rects * 16) == cudaSuccess &&
             cudaMalloc(&b->d_overlay_count, (size_t)b->num_obs * 4) == cudaSuccess &&
             cudaMemset(b->d_overlay_count, 0, (size_t)b->num_obs * 4) == cudaSuccess;
    if (ok) ok = cudaMemset(b->d_env_blocks, 0, blocks_bytes) == cudaSuccess &&
                 cudaMemset(b->d_status, 0, 16) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        mv_destroy(b);
        return MV_ERR_OUT_OF_MEMORY;
    }
    *out = b;
    return MV_OK;
}

int mv_upload_worlds(mv_batch *b, int env_begin, int env_count, const uint8_t *d_grid, const mv_box *d_boxes,
                     const int32_t *d_box_count, const uint8_t *d_palette, void *cuda_stream) {
    if (!b || env_begin < 0 || env_count < 0 || (int64_t)env_begin + env_count > b->desc.num_envs)
        return MV_ERR_INVALID_ARG;
    return upload_worlds(b, env_begin, nullptr, env_count, d_grid, d_boxes, d_box_count, d_palette,
                         static_cast<cudaStream_t>(cuda_stream));
}

int mv_upload_worlds_at(mv_batch *b, int env_count, const int32_t *h_env_index, const uint8_t *d_grid,
                        const mv_box *d_boxes, const int32_t *d_box_count, const uint8_t *d_palette,
                        void *cuda_stream) {
    if (!b || env_count < 0 || env_count > b->desc.num_envs || (env_count > 0 && !h_env_index))
        return MV_ERR_INVALID_ARG;
    for (int i = 0; i < env_count; ++i)          // strictly increasing: in range and no env written twice
        if (h_env_index[i] < 0 || h_env_index[i] >= b->desc.num_envs || (i > 0 && h_env_index[i] <= h_env_index[i - 1]))
            return MV_ERR_INVALID_ARG;
    return upload_worlds(b, 0, h_env_index, env_count, d_grid, d_boxes, d_box_count, d_palette,
                         static_cast<cudaStream_t>(cuda_stream));
}

int mv_set_cameras(mv_batch *b, const mv_camera *d_cams, void *cuda_stream) {
    if (!b || !d_cams) return MV_ERR_INVALID_ARG;
    DeviceGuard g(b->desc.device);
    if (!g.ok) return MV_ERR_CUDA;
    return launch_cameras(b, d_cams, static_cast<cudaStream_t>(cuda_stream));
}

int mv_set_overlays(mv_batch *b, const mv_overlay_rect *d_rects, const int32_t *d_count, void *cuda_stream) {
    if (!b || (d_rects && !d_count)) return MV_ERR_INVALID_ARG;
    const int m = b->desc.max_overlay_rects;
    if (m == 0) return d_rects ? MV_ERR_INVALID_ARG : MV_OK;
    if (d_rects && !aligned16(d_rects)) return MV_ERR_INVALID_ARG;
    DeviceGuard g(b->desc.device);
    if (!g.ok) return MV_ERR_CUDA;
    const int n = b->num_obs * (m + 1);
    copy_overlays_kernel<<<(n + 255) / 256, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        reinterpret_cast<const int4 *>(d_rects), d_count, b->d_overlay, b->d_overlay_count, b->num_obs, m);
    b->launches++;
    MV_CUDA(b, cudaGetLastError());
    return MV_OK;
}

int mv_move_agents(mv_batch *b, mv_camera *d_cams_inout, const mv_agent_move *d_moves, const mv_body_shape *shape,
                   void *cuda_stream) {
    if (!b || !d_cams_inout || !d_moves || !aligned16(d_moves)) return MV_ERR_INVALID_ARG;
    mv_body_shape sh = {0.25f, 0.75f, 0.25f, 1.0f};
    if (shape) sh = *shape;
    if (!(sh.half_width >= 0.0f) || !(sh.below_eye >= 0.0f) || !(sh.above_eye >= 0.0f) || !(sh.max_pitch >= 0.0f) ||
        !(sh.half_width < 16.0f) || !(sh.below_eye < 16.0f) || !(sh.above_eye < 16.0f))
        return MV_ERR_INVALID_ARG;
    if (b->missing_grid > 0) return MV_ERR_NOT_READY;
    DeviceGuard g(b->desc.device);
    if (!g.ok) return MV_ERR_CUDA;
    const int n = b->num_obs;
    move_agents_kernel<<<(n + 127) / 128, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        reinterpret_cast<int32_t *>(d_cams_inout), reinterpret_cast<const float4 *>(d_moves), b->d_cams,
        b->d_env_blocks, b->lay, n, b->desc.agents_per_env, b->desc.grid_x, b->desc.grid_y, b->desc.grid_z,
        b->desc.max_boxes, sh.half_width, sh.below_eye, sh.above_eye, sh.max_pitch, b->kr, b->ku, b->d_status);
    b->launches++;
    MV_CUDA(b, cudaGetLastError());
    b->has_cams = true;
    return MV_OK;
}

int mv_merge_voxels(mv_batch *b, int env_begin, int env_count, mv_box *d_boxes_out, int32_t *d_count_out,
                    int max_out, void *cuda_stream) {
    if (!b || env_begin < 0 || env_count < 0 || (int64_t)env_begin + env_count > b->desc.num_envs || !d_boxes_out ||
        !d_count_out || max_out < 1 || !aligned16(d_boxes_out))
        return MV_ERR_INVALID_ARG;
    for (int e = env_begin; e < env_begin + env_count; ++e)
        if (!b->has_grid[e]) return MV_ERR_NOT_READY;
    if (env_count == 0) return MV_OK;
    DeviceGuard g(b->desc.device);
    if (!g.ok) return MV_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t words = b->nvox / 32;
    if (!b->d_covered) {
        size_t chunk = kMergeScratchBytes / (words * 4 * 2);       // coverage bits + x-packed occupancy per env
        chunk = chunk < 1 ? 1 : (chunk > (size_t)b->desc.num_envs ? (size_t)b->desc.num_envs : chunk);
        MV_CUDA(b, cudaMalloc(&b->d_covered, chunk * words * 4 * 2));
        b->merge_chunk = (int)chunk;
    }
    const int kMergeChunk = b->merge_chunk;
    for (int e0 = 0; e0 < env_count; e0 += kMergeChunk) {
        const int n = env_count - e0 < kMergeChunk ? env_count - e0 : kMergeChunk;
        uint32_t *occx = b->d_covered + (size_t)kMergeChunk * words;
        MV_CUDA(b, cudaMemsetAsync(b->d_covered, 0, (size_t)n * words * 4, s));
        xpack_kernel<<<(unsigned)(((size_t)n * words + 255) / 256), 256, 0, s>>>(
            b->d_env_blocks, b->lay, env_begin + e0, n, b->desc.grid_x, b->desc.grid_y, b->desc.grid_z, occx);
        b->launches++;
        MV_CUDA(b, cudaGetLastError());
        merge_voxels_kernel<<<(n * 32 + 127) / 128, 128, 0, s>>>(
            occx, b->d_mat, b->lay, env_begin + e0, n, b->desc.grid_x, b->desc.grid_y, b->desc.grid_z,
            b->d_covered, reinterpret_cast<uint4 *>(d_boxes_out + (size_t)e0 * max_out), d_count_out + e0, max_out);
        b->launches++;
        MV_CUDA(b, cudaGetLastError());
    }
    return MV_OK;
}

int mv_render_batch(mv_batch *b, uint8_t *d_rgb, float *d_depth, void *cuda_stream) {
    if (!b || !d_rgb || !d_depth || !aligned16(d_rgb) || !aligned16(d_depth)) return MV_ERR_INVALID_ARG;
    if (b->missing_grid > 0 || b->missing_palette > 0 || !b->has_cams) return MV_ERR_NOT_READY;
    DeviceGuard g(b->desc.device);
    if (!g.ok) return MV_ERR_CUDA;
    return launch_render(b, d_rgb, d_depth, 0, b->num_obs, static_cast<cudaStream_t>(cuda_stream));
}

int mv_step_host(mv_batch *b, const mv_camera *h_cams, const mv_box *h_boxes, const int32_t *h_box_count,
                 uint8_t *h_rgb, float *h_depth, void *cuda_stream) {
    if (!b || !h_cams || !h_rgb || !h_depth) return MV_ERR_INVALID_ARG;
    if (h_boxes && (!h_box_count || b->desc.max_boxes == 0)) return MV_ERR_INVALID_ARG;
    if (b->missing_grid > 0 || b->missing_palette > 0) return MV_ERR_NOT_READY;
    DeviceGuard g(b->desc.device);
    if (!g.ok) return MV_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t px = (size_t)b->desc.width * b->desc.height;
    const int E = b->desc.num_envs, O = b->num_obs;
    if (!b->host_ready) {
        int r = alloc_host_step(b);
        if (r != MV_OK) return r;
    }
    MV_CUDA(b, cudaMemcpyAsync(b->d_cam_in, h_cams, (size_t)O * sizeof(mv_camera), cudaMemcpyHostToDevice, s));
    if (h_boxes) {
        MV_CUDA(b, cudaMemcpyAsync(b->d_box_in, h_boxes, (size_t)E * b->desc.max_boxes * sizeof(mv_box),
                                   cudaMemcpyHostToDevice, s));
        MV_CUDA(b, cudaMemcpyAsync(b->d_count_in, h_box_count, (size_t)E * sizeof(int32_t), cudaMemcpyHostToDevice, s));
        int r = launch_boxes(b, 0, nullptr, E, b->d_box_in, b->d_count_in, s);
        if (r != MV_OK) return r;
    }
    int r = launch_cameras(b, b->d_cam_in, s);
    if (r != MV_OK) return r;
    // render chunk by chunk; each chunk's frames start their trip to the host while the next renders
    // (chunks are whole environments, as the render launch wants when one CTA renders an env)
    const int A = b->desc.agents_per_env;
    const int chunks = E < kHostChunks ? 1 : kHostChunks;
    for (int c = 0; c < chunks; ++c) {
        const int o0 = (int)((int64_t)E * c / chunks) * A, o1 = (int)((int64_t)E * (c + 1) / chunks) * A;
        r = launch_render(b, b->d_rgb, b->d_depth, o0, o1 - o0, s);
        if (r != MV_OK) return r;
        MV_CUDA(b, cudaEventRecord(b->ev_chunk[c], s));
        MV_CUDA(b, cudaStreamWaitEvent(b->copy_stream, b->ev_chunk[c], 0));
        MV_CUDA(b, cudaMemcpyAsync(h_rgb + (size_t)o0 * px * 3, b->d_rgb + (size_t)o0 * px * 3,
                                   (size_t)(o1 - o0) * px * 3, cudaMemcpyDeviceToHost, b->copy_stream));
        MV_CUDA(b, cudaMemcpyAsync(h_depth + (size_t)o0 * px, b->d_depth + (size_t)o0 * px,
                                   (size_t)(o1 - o0) * px * 4, cudaMemcpyDeviceToHost, b->copy_stream));
    }
    MV_CUDA(b, cudaEventRecord(b->ev_done, b->copy_stream));
    MV_CUDA(b, cudaStreamWaitEvent(s, b->ev_done, 0));
    return finish_host_step(b, s);
}

int mv_step_host_static(mv_batch *b, const mv_camera *h_cams, uint8_t *h_rgb, float *h_depth,
                        void *cuda_stream) {
    if (!b || !h_cams || !h_rgb || !h_depth) return MV_ERR_INVALID_ARG;
    if (b->missing_grid > 0 || b->missing_palette > 0) return MV_ERR_NOT_READY;
    const size_t px = (size_t)b->desc.width * b->desc.height;
    const size_t O = (size_t)b->num_obs;
    // layout inside the scratch array: depth | rgb | cameras, each 256-byte aligned
    const size_t depth_bytes = (O * px * 4 + 255) / 256 * 256;
    const size_t rgb_bytes = (O * px * 3 + 255) / 256 * 256;
    const size_t cam_bytes = O * sizeof(mv_camera);
    if (depth_bytes + rgb_bytes + cam_bytes > (size_t)MV_STATIC_SCRATCH_BYTES) return MV_ERR_UNSUPPORTED;
    DeviceGuard g(b->desc.device);
    if (!g.ok) return MV_ERR_CUDA;
    unsigned char *scratch = nullptr;
    int r = static_scratch_for_device(b, b->desc.device, &scratch);
    if (r != MV_OK) return r;
    float *d_depth = reinterpret_cast<float *>(scratch);
    uint8_t *d_rgb = scratch + depth_bytes;
    mv_camera *d_cams = reinterpret_cast<mv_camera *>(scratch + depth_bytes + rgb_bytes);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    // nothing in the scratch has to start at zero: the cameras are overwritten by the copy
    // below and the render kernel writes every byte of both frame buffers
    MV_CUDA(b, cudaMemcpyAsync(d_cams, h_cams, cam_bytes, cudaMemcpyHostToDevice, s));
    r = launch_cameras(b, d_cams, s);
    if (r != MV_OK) return r;
    r = launch_render(b, d_rgb, d_depth, 0, b->num_obs, s);
    if (r != MV_OK) return r;
    MV_CUDA(b, cudaMemcpyAsync(h_rgb, d_rgb, O * px * 3, cudaMemcpyDeviceToHost, s));
    MV_CUDA(b, cudaMemcpyAsync(h_depth, d_depth, O * px * 4, cudaMemcpyDeviceToHost, s));
    return finish_host_step(b, s);
}

int mv_query_status(mv_batch *b, int clear, void *cuda_stream) {
    if (!b) return MV_ERR_INVALID_ARG;
    DeviceGuard g(b->desc.device);
    if (!g.ok) return MV_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    uint32_t word = 0;
    MV_CUDA(b, cudaMemcpyAsync(&word, b->d_status, 4, cudaMemcpyDeviceToHost, s));
    if (clear) MV_CUDA(b, cudaMemsetAsync(b->d_status, 0, 4, s));
    MV_CUDA(b, cudaStreamSynchronize(s));
    if (word & kFlagTimeout) return MV_ERR_DEVICE_TIMEOUT;
    return (int)word;
}

int64_t mv_launch_count(const mv_batch *b) { return b ? b->launches : 0; }

int mv_debug_occupancy_in_global(mv_batch *b, int on) {
    if (!b) return MV_ERR_INVALID_ARG;
    if (!on && !b->occ_fits_shared) return MV_ERR_UNSUPPORTED;
    b->occ_shared = !on;
    return MV_OK;
}

int mv_debug_agents_per_cta(mv_batch *b, int agents_per_cta) {
    if (!b) return MV_ERR_INVALID_ARG;
    const int A = b->desc.agents_per_env;
    int apc = agents_per_cta == 0 ? b->auto_agents_per_cta : agents_per_cta;
    if (apc != 1 && apc != A) return MV_ERR_INVALID_ARG;
    const mv_batch::Smem m = smem_layout(b, apc);
    if ((int)(m.bytes - b->lay.occ_bytes) > b->smem_max) return MV_ERR_UNSUPPORTED;
    b->occ_fits_shared = (int)m.bytes <= b->smem_max;
    if (!b->occ_fits_shared) b->occ_shared = false;
    b->smem = m;
    b->agents_per_cta = apc;
    b->threads = pick_threads(b, apc);
    return MV_OK;
}

int mv_debug_staging(mv_batch *b, int skip_staging, int wait_polls) {
    if (!b || wait_polls < 1 || wait_polls > (1 << 24)) return MV_ERR_INVALID_ARG;
    b->skip_staging = skip_staging ? 1 : 0;
    b->wait_polls = wait_polls;
    return MV_OK;
}

int mv_destroy(mv_batch *b) {
    if (!b) return MV_OK;
    int rc = MV_OK;
    {
        DeviceGuard g(b->desc.device);
        if (g.ok) {
            if (cudaDeviceSynchronize() != cudaSuccess) rc = MV_ERR_CUDA;
            cudaFree(b->d_env_blocks); cudaFree(b->d_mat); cudaFree(b->d_cams); cudaFree(b->d_status);
            cudaFree(b->d_overlay); cudaFree(b->d_overlay_count); cudaFree(b->d_covered); cudaFree(b->d_env_index);
            free_host_step(b);
            cudaGetLastError();
        }
    }
    delete b;
    return rc;
}

}  // extern "C"
