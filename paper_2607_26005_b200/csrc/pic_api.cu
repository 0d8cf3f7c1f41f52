// C ABI of the rasterizer library: scene management, argument validation, launches.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

#include "../../include/pictura.h"
#include "pic_types.h"

namespace pic {
size_t max_smem_bytes();
cudaError_t configure_kernels();
cudaError_t launch_setup(const RenderParams& P, int n_agents, const float* poses, float* state, const float* actions,
                         const float* dims, const uint8_t* active, const uint8_t* agent_cls, AgentGeom* agents_out, ViewCam* cams_out,
                         float* tables, uint32_t* status, float dt, float wheelbase, float v_max, cudaStream_t stream);
cudaError_t launch_render(const RenderParams& P, long long n_views, bool brute, int sm_count, cudaStream_t stream);
cudaError_t launch_colour(const RenderParams& P, long long n_views, bool antialias, cudaStream_t stream);
size_t survivor_bytes_per_tile();
}  // namespace pic

namespace {

constexpr float kDt = 0.1f, kWheelbase = 2.8f, kVMax = 30.0f;
constexpr int kMaxTimed = 1024;

thread_local char g_err[512] = "";

pic_status fail(pic_status st, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return st;
}

}  // namespace

namespace pic {
// lets the other translation units of the library report through pic_last_error()
void set_last_error(const char* msg) { snprintf(g_err, sizeof(g_err), "%s", msg); }
}  // namespace pic

namespace {

#define CUDA_TRY(expr)                                                                                   \
    do {                                                                                                 \
        cudaError_t _e = (expr);                                                                         \
        if (_e != cudaSuccess)                                                                           \
            return fail(_e == cudaErrorMemoryAllocation ? PIC_ERR_OOM : PIC_ERR_CUDA, "%s: %s", #expr,   \
                        cudaGetErrorString(_e));                                                         \
    } while (0)

}  // namespace

struct pic_scene {
    int E = 0, A = 0, K = 0, H = 0, W = 0;
    float near_z = 0, far_z = 0;
    int M = 0;
    uint8_t cls_agent = 0, cls_sky = 0, cls_ground = 0;
    int device = 0;
    // device memory owned by the scene
    int32_t* d_env_map = nullptr;
    pic::MapInfo* d_maps = nullptr;
    pic::MapInfo* d_env_maps = nullptr;   // [E]
    pic::Node* d_groups = nullptr;
    pic::Node* d_leaves = nullptr;
    pic::Prim* d_prims = nullptr;
    uint32_t* d_cell_start = nullptr;
    pic::Prim* d_grid_prims = nullptr;
    pic::Node* d_large_leaves = nullptr;
    pic::AgentGeom* d_agents = nullptr;
    pic::ViewCam* d_cams = nullptr;   // [E*A*K]
    uint32_t* d_overflow = nullptr;   // [1 + E*A*K*tiles] tiles handed from the render kernel to the cooperative kernel
    uint2* d_surv = nullptr;          // per tile: survivors of the cull kernel, read by the render kernel
    int sm_count = 0;
    float* d_tables = nullptr;        // per-camera ray and background tables, K*(W+3H) words
    float* d_state = nullptr;       // [E*A*4]
    float* d_dims = nullptr;        // [E*A*3]
    uint8_t* d_active = nullptr;    // [E*A]
    bool have_active = false;
    uint8_t* d_agent_cls = nullptr; // [E*A] class of each agent's box
    bool have_agent_cls = false;
    uint32_t* d_status = nullptr;
    uint8_t* d_palette = nullptr;   // [256][3] RGB of every class, for the colour output
    // staging for pic_render_host
    float* d_in_poses = nullptr;
    float* d_in_dims = nullptr;
    uint8_t* d_in_active = nullptr;
    uint8_t* d_out_class = nullptr;
    uint16_t* d_out_depth = nullptr;
    // options
    bool brute = false;
    float* depth32 = nullptr;
    unsigned long long* counters = nullptr;
    uint32_t* occlusion = nullptr;
    long long view_first = 0, view_count = 0;
    int debug_flags = 0;
    bool out_relative = false;
    bool timing = false;
    cudaEvent_t* ev = nullptr;      // 2 * kMaxTimed events
    int n_timed = 0;
    size_t n_prims = 0, n_leaves = 0, n_groups = 0;
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

void free_scene(pic_scene* s) {
    cudaFree(s->d_env_map); cudaFree(s->d_env_maps); cudaFree(s->d_maps); cudaFree(s->d_groups); cudaFree(s->d_leaves); cudaFree(s->d_prims); cudaFree(s->d_cell_start); cudaFree(s->d_grid_prims); cudaFree(s->d_large_leaves);
    cudaFree(s->d_agents); cudaFree(s->d_cams); cudaFree(s->d_overflow); cudaFree(s->d_surv); cudaFree(s->d_tables); cudaFree(s->d_state); cudaFree(s->d_dims); cudaFree(s->d_active); cudaFree(s->d_agent_cls); cudaFree(s->d_status); cudaFree(s->d_palette);
    cudaFree(s->d_in_poses); cudaFree(s->d_in_dims); cudaFree(s->d_in_active); cudaFree(s->d_out_class);
    cudaFree(s->d_out_depth);
    if (s->ev) {
        for (int i = 0; i < 2 * kMaxTimed; ++i) if (s->ev[i]) cudaEventDestroy(s->ev[i]);
        delete[] s->ev;
    }
    delete s;
}

pic_status fill_params(const pic_scene* s, const pic_camera* rig, uint8_t* out_class, uint16_t* out_depth,
                       pic::RenderParams& P, bool colour = false) {
    if (!rig) return fail(PIC_ERR_INVALID_ARG, "rig is NULL");
    if (!colour && (!out_class || !out_depth)) return fail(PIC_ERR_INVALID_ARG, "output pointer is NULL");
    if ((reinterpret_cast<uintptr_t>(out_class) & 15u) || (reinterpret_cast<uintptr_t>(out_depth) & 15u))
        return fail(PIC_ERR_INVALID_ARG, "output pointers must be 16-byte aligned");
    std::memset(&P, 0, sizeof(P));
    P.E = s->E; P.A = s->A; P.K = s->K; P.H = s->H; P.W = s->W;
    P.tiles_x = (s->W + pic::TILE - 1) / pic::TILE;
    P.tiles_y = (s->H + pic::TILE - 1) / pic::TILE;
    P.near_z = s->near_z; P.far_z = s->far_z;
    P.w_near = 1.0f / s->near_z; P.w_far = 1.0f / s->far_z;
    P.cls_agent = s->cls_agent; P.cls_sky = s->cls_sky; P.cls_ground = s->cls_ground;
    P.env_map = s->d_env_map; P.env_maps = s->d_env_maps; P.maps = s->d_maps; P.groups = s->d_groups; P.leaves = s->d_leaves; P.prims = s->d_prims;
    P.cell_start = s->d_cell_start; P.grid_prims = s->d_grid_prims; P.large_leaves = s->d_large_leaves;
    P.agents = s->d_agents;
    P.cams = s->d_cams;
    P.overflow = s->d_overflow;
    P.surv = s->d_surv;
    P.palette = s->d_palette;
    P.status = s->d_status;
    P.rig.ray_x = s->d_tables;
    P.rig.ray_y = P.rig.ray_x + (size_t)s->K * s->W;
    P.rig.bg_z = P.rig.ray_y + (size_t)s->K * s->H;
    P.rig.bg_cls = reinterpret_cast<const uint32_t*>(P.rig.bg_z + (size_t)s->K * s->H);
    P.out_class = out_class; P.out_depth = out_depth; P.out_depth32 = s->depth32; P.counters = s->counters; P.occlusion = s->occlusion;
    P.view_first = 0;
    P.debug_flags = s->debug_flags;
    for (int k = 0; k < s->K; ++k) {
        const pic_camera& c = rig[k];
        const float vals[7] = {c.mount_x, c.mount_y, c.mount_z, c.yaw, c.pitch, c.fx, c.fy};
        for (float v : vals)
            if (!std::isfinite(v)) return fail(PIC_ERR_INVALID_ARG, "camera %d has a non-finite field", k);
        if (!(c.fx > 0.f) || !(c.fy > 0.f)) return fail(PIC_ERR_INVALID_ARG, "camera %d: focal lengths must be positive", k);
        pic::CamConst& o = P.cam[k];
        o.mx = c.mount_x; o.my = c.mount_y; o.mz = c.mount_z;
        o.cpsi = (float)std::cos((double)c.yaw); o.spsi = (float)std::sin((double)c.yaw);
        o.cphi = (float)std::cos((double)c.pitch); o.sphi = (float)std::sin((double)c.pitch);
        o.fx = c.fx; o.fy = c.fy;
    }
    return PIC_OK;
}

}  // namespace

extern "C" {

const char* pic_last_error(void) { return g_err; }

int32_t pic_version(void) { return 100; }

pic_status pic_scene_create(const pic_scene_desc* d, pic_scene** out) {
    if (!d || !out) return fail(PIC_ERR_INVALID_ARG, "desc or out is NULL");
    *out = nullptr;
    if (d->size != sizeof(pic_scene_desc))
        return fail(PIC_ERR_INVALID_ARG, "desc->size is %u, this library expects %zu", d->size, sizeof(pic_scene_desc));
    if (d->E <= 0 || d->A <= 0 || d->K <= 0 || d->H <= 0 || d->W <= 0)
        return fail(PIC_ERR_SHAPE, "E, A, K, H, W must be positive");
    if (d->K > pic::MAX_CAMS) return fail(PIC_ERR_SHAPE, "at most %d cameras per rig", pic::MAX_CAMS);
    if (d->H > 16384 || d->W > 16384) return fail(PIC_ERR_SHAPE, "images larger than 16384 pixels per side are not supported");
    if ((long long)d->E * d->A > (1LL << 28)) return fail(PIC_ERR_SHAPE, "E*A too large");
    if (!(d->near_z > 0.f) || !(d->far_z > d->near_z) || !std::isfinite(d->far_z))
        return fail(PIC_ERR_INVALID_ARG, "need 0 < near_z < far_z < inf");
    if (d->num_maps <= 0) return fail(PIC_ERR_SHAPE, "num_maps must be positive");
    if (!d->map_tri_offset) return fail(PIC_ERR_INVALID_ARG, "map_tri_offset is NULL");
    if (d->map_tri_offset[0] != 0) return fail(PIC_ERR_SHAPE, "map_tri_offset[0] must be 0");
    for (int m = 0; m < d->num_maps; ++m)
        if (d->map_tri_offset[m + 1] < d->map_tri_offset[m]) return fail(PIC_ERR_SHAPE, "map_tri_offset must be non-decreasing");
    const int64_t n_tri = d->map_tri_offset[d->num_maps];
    if (n_tri > 0 && (!d->tri_xyz || !d->tri_class)) return fail(PIC_ERR_INVALID_ARG, "triangle arrays are NULL");
    for (int64_t i = 0; i < 9 * n_tri; ++i)
        if (!std::isfinite(d->tri_xyz[i])) return fail(PIC_ERR_INVALID_ARG, "triangle %lld has a non-finite coordinate", (long long)(i / 9));
    if (d->env_map_id) {
        for (int e = 0; e < d->E; ++e)
            if (d->env_map_id[e] < 0 || d->env_map_id[e] >= d->num_maps) return fail(PIC_ERR_SHAPE, "env_map_id[%d] out of range", e);
    } else if (d->num_maps != 1 && d->num_maps != d->E) {
        return fail(PIC_ERR_SHAPE, "env_map_id is NULL but num_maps is neither 1 nor E");
    }
    int n_dev = 0;
    CUDA_TRY(cudaGetDeviceCount(&n_dev));
    if (d->device < 0 || d->device >= n_dev) return fail(PIC_ERR_INVALID_ARG, "device %d does not exist", d->device);
    DeviceGuard guard(d->device);
    if (!guard.ok) return fail(PIC_ERR_CUDA, "cannot select device %d", d->device);
    cudaDeviceProp prop;
    CUDA_TRY(cudaGetDeviceProperties(&prop, d->device));
    if (prop.major < 10) return fail(PIC_ERR_CUDA, "device %d is sm_%d%d; this library is built for sm_100a only", d->device, prop.major, prop.minor);
    if ((size_t)prop.sharedMemPerBlockOptin < pic::max_smem_bytes())
        return fail(PIC_ERR_CUDA, "device offers %zu bytes of shared memory per block, %zu needed", (size_t)prop.sharedMemPerBlockOptin, pic::max_smem_bytes());
    CUDA_TRY(pic::configure_kernels());

    char err[256] = "";
    if (d->tri_vis_cos)
        for (int64_t i = 0; i < n_tri; ++i)
            if (!(d->tri_vis_cos[i] >= 0.f) || d->tri_vis_cos[i] > 1.f) return fail(PIC_ERR_INVALID_ARG, "tri_vis_cos[%lld] is not in [0, 1]", (long long)i);
    pic::HostHierarchy* hh = pic::build_hierarchy(d->num_maps, d->map_tri_offset, d->tri_xyz, d->tri_class, d->tri_vis_cos, d->A, err, sizeof(err));
    if (!hh) return fail(PIC_ERR_SHAPE, "%s", err);

    pic_scene* s = new (std::nothrow) pic_scene();
    if (!s) { pic::free_hierarchy(hh); return fail(PIC_ERR_OOM, "host allocation failed"); }
    s->E = d->E; s->A = d->A; s->K = d->K; s->H = d->H; s->W = d->W;
    s->near_z = d->near_z; s->far_z = d->far_z; s->M = d->num_maps;
    s->cls_agent = d->agent_class; s->cls_sky = d->sky_class; s->cls_ground = d->ground_class;
    s->device = d->device;
    s->sm_count = prop.multiProcessorCount;

    size_t np, nl, ng, nm;
    const pic::Prim* prims = pic::hierarchy_prims(hh, &np);
    const pic::Node* leaves = pic::hierarchy_leaves(hh, &nl);
    const pic::Node* groups = pic::hierarchy_groups(hh, &ng);
    const pic::MapInfo* maps = pic::hierarchy_maps(hh, &nm);
    size_t ncs, ngp, nll;
    const uint32_t* cell_start = pic::hierarchy_cell_start(hh, &ncs);
    const pic::Prim* grid_prims = pic::hierarchy_grid_prims(hh, &ngp);
    const pic::Node* large_leaves = pic::hierarchy_large_leaves(hh, &nll);
    s->n_prims = np; s->n_leaves = nl; s->n_groups = ng;
    const size_t n_agents = (size_t)d->E * d->A;
    int32_t* env_map = new (std::nothrow) int32_t[d->E];
    if (!env_map) { pic::free_hierarchy(hh); free_scene(s); return fail(PIC_ERR_OOM, "host allocation failed"); }
    for (int e = 0; e < d->E; ++e) env_map[e] = d->env_map_id ? d->env_map_id[e] : (d->num_maps == 1 ? 0 : e);

    cudaError_t ce = cudaSuccess;
    auto dmalloc = [&](void** p, size_t bytes) { if (ce == cudaSuccess) ce = cudaMalloc(p, bytes ? bytes : 16); };
    auto upload = [&](void* dst, const void* src, size_t bytes) {
        if (ce == cudaSuccess && bytes) ce = cudaMemcpy(dst, src, bytes, cudaMemcpyHostToDevice);
    };
    dmalloc((void**)&s->d_env_map, sizeof(int32_t) * d->E);
    dmalloc((void**)&s->d_maps, sizeof(pic::MapInfo) * nm);
    dmalloc((void**)&s->d_env_maps, sizeof(pic::MapInfo) * d->E);
    dmalloc((void**)&s->d_groups, sizeof(pic::Node) * ng);
    dmalloc((void**)&s->d_leaves, sizeof(pic::Node) * nl);
    dmalloc((void**)&s->d_prims, sizeof(pic::Prim) * np);
    dmalloc((void**)&s->d_cell_start, sizeof(uint32_t) * ncs);
    dmalloc((void**)&s->d_grid_prims, sizeof(pic::Prim) * ngp);
    dmalloc((void**)&s->d_large_leaves, sizeof(pic::Node) * nll);
    dmalloc((void**)&s->d_agents, sizeof(pic::AgentGeom) * n_agents);
    dmalloc((void**)&s->d_cams, sizeof(pic::ViewCam) * n_agents * d->K);
    dmalloc((void**)&s->d_overflow, sizeof(uint32_t) * (1 + (size_t)n_agents * d->K * ((d->W + pic::TILE - 1) / pic::TILE) * ((d->H + pic::TILE - 1) / pic::TILE)));
    dmalloc((void**)&s->d_surv, pic::survivor_bytes_per_tile() * (size_t)n_agents * d->K * ((d->W + pic::TILE - 1) / pic::TILE) * ((d->H + pic::TILE - 1) / pic::TILE));
    dmalloc((void**)&s->d_tables, sizeof(float) * (size_t)d->K * ((size_t)d->W + 3 * (size_t)d->H));
    dmalloc((void**)&s->d_state, sizeof(float) * 4 * n_agents);
    dmalloc((void**)&s->d_dims, sizeof(float) * 3 * n_agents);
    dmalloc((void**)&s->d_active, n_agents);
    dmalloc((void**)&s->d_agent_cls, n_agents);
    dmalloc((void**)&s->d_status, sizeof(uint32_t));
    dmalloc((void**)&s->d_palette, 768);
    upload(s->d_env_map, env_map, sizeof(int32_t) * d->E);
    upload(s->d_maps, maps, sizeof(pic::MapInfo) * nm);
    {
        pic::MapInfo* per_env = new (std::nothrow) pic::MapInfo[d->E];
        if (!per_env) { if (ce == cudaSuccess) ce = cudaErrorMemoryAllocation; }
        else {
            for (int e = 0; e < d->E; ++e) per_env[e] = maps[env_map[e]];
            upload(s->d_env_maps, per_env, sizeof(pic::MapInfo) * d->E);
            delete[] per_env;
        }
    }
    upload(s->d_groups, groups, sizeof(pic::Node) * ng);
    upload(s->d_leaves, leaves, sizeof(pic::Node) * nl);
    upload(s->d_prims, prims, sizeof(pic::Prim) * np);
    upload(s->d_cell_start, cell_start, sizeof(uint32_t) * ncs);
    upload(s->d_grid_prims, grid_prims, sizeof(pic::Prim) * ngp);
    upload(s->d_large_leaves, large_leaves, sizeof(pic::Node) * nll);
    if (ce == cudaSuccess) ce = cudaMemset(s->d_status, 0, sizeof(uint32_t));
    if (ce == cudaSuccess) {          // until pic_set_palette: class c is the grey (c, c, c)
        uint8_t grey[768];
        for (int c = 0; c < 256; ++c) grey[3 * c] = grey[3 * c + 1] = grey[3 * c + 2] = (uint8_t)c;
        ce = cudaMemcpy(s->d_palette, grey, 768, cudaMemcpyHostToDevice);
    }
    if (ce == cudaSuccess) ce = cudaMemset(s->d_state, 0, sizeof(float) * 4 * n_agents);
    if (ce == cudaSuccess) ce = cudaMemset(s->d_dims, 0, sizeof(float) * 3 * n_agents);
    if (ce == cudaSuccess) ce = cudaMemset(s->d_active, 1, n_agents);
    delete[] env_map;
    pic::free_hierarchy(hh);
    if (ce != cudaSuccess) {
        free_scene(s);
        return fail(ce == cudaErrorMemoryAllocation ? PIC_ERR_OOM : PIC_ERR_CUDA, "scene allocation/upload: %s", cudaGetErrorString(ce));
    }
    *out = s;
    return PIC_OK;
}

pic_status pic_map_stats(const pic_scene_desc* d, int64_t out[8]) {
    if (!d || !out) return fail(PIC_ERR_INVALID_ARG, "desc or out is NULL");
    if (d->size != sizeof(pic_scene_desc)) return fail(PIC_ERR_INVALID_ARG, "desc->size mismatch");
    if (d->num_maps <= 0 || !d->map_tri_offset || d->map_tri_offset[0] != 0) return fail(PIC_ERR_SHAPE, "bad map offsets");
    for (int m = 0; m < d->num_maps; ++m)
        if (d->map_tri_offset[m + 1] < d->map_tri_offset[m]) return fail(PIC_ERR_SHAPE, "map_tri_offset must be non-decreasing");
    if (d->map_tri_offset[d->num_maps] > 0 && (!d->tri_xyz || !d->tri_class)) return fail(PIC_ERR_INVALID_ARG, "triangle arrays are NULL");
    char err[256] = "";
    pic::HostHierarchy* hh = pic::build_hierarchy(d->num_maps, d->map_tri_offset, d->tri_xyz, d->tri_class, d->tri_vis_cos, d->A > 0 ? d->A : 0, err, sizeof(err));
    if (!hh) return fail(PIC_ERR_SHAPE, "%s", err);
    size_t np, nl, ng, nm;
    const pic::Prim* prims = pic::hierarchy_prims(hh, &np);
    const pic::Node* leaves = pic::hierarchy_leaves(hh, &nl);
    const pic::Node* groups = pic::hierarchy_groups(hh, &ng);
    pic::hierarchy_maps(hh, &nm);
    int64_t quads = 0, largest = 0, prim_out = 0, leaf_out = 0, tris = 0;
    for (size_t i = 0; i < np; ++i) { const bool q = prims[i].flags & 1u; quads += q; tris += q ? 2 : 1; }
    for (size_t l = 0; l < nl; ++l) {
        const pic::Node& lf = leaves[l];
        if ((int64_t)lf.count > largest) largest = lf.count;
        for (uint32_t k = 0; k < lf.count; ++k) {
            const pic::Prim& p = prims[lf.first + k];
            const int nv = (p.flags & 1u) ? 4 : 3;
            bool inside = true;
            for (int v = 0; v < nv; ++v)
                for (int c = 0; c < 3; ++c)
                    inside = inside && p.v[3 * v + c] >= lf.lo[c] && p.v[3 * v + c] <= lf.hi[c];
            prim_out += !inside;
        }
    }
    for (size_t g = 0; g < ng; ++g) {
        const pic::Node& gr = groups[g];
        for (uint32_t k = 0; k < gr.count; ++k) {
            const pic::Node& lf = leaves[gr.first + k];
            bool inside = true;
            for (int c = 0; c < 3; ++c) inside = inside && lf.lo[c] >= gr.lo[c] && lf.hi[c] <= gr.hi[c];
            leaf_out += !inside;
        }
    }
    out[0] = (int64_t)np; out[1] = quads; out[2] = (int64_t)nl; out[3] = (int64_t)ng; out[4] = largest;
    out[5] = prim_out; out[6] = leaf_out; out[7] = tris;
    pic::free_hierarchy(hh);
    return PIC_OK;
}

pic_status pic_scene_destroy(pic_scene* s) {
    if (!s) return PIC_OK;
    DeviceGuard guard(s->device);
    cudaDeviceSynchronize();
    free_scene(s);
    return PIC_OK;
}

pic_status pic_scene_set_option(pic_scene* s, int32_t option, uint64_t value) {
    if (!s) return fail(PIC_ERR_INVALID_ARG, "scene is NULL");
    switch (option) {
        case PIC_OPT_BRUTE_FORCE: s->brute = value != 0; return PIC_OK;
        case PIC_OPT_DEPTH32: s->depth32 = reinterpret_cast<float*>(static_cast<uintptr_t>(value)); return PIC_OK;
        case PIC_OPT_COUNTERS: s->counters = reinterpret_cast<unsigned long long*>(static_cast<uintptr_t>(value)); return PIC_OK;
        case PIC_OPT_OCCLUSION: s->occlusion = reinterpret_cast<uint32_t*>(static_cast<uintptr_t>(value)); return PIC_OK;
        case PIC_OPT_VIEW_FIRST:
            if (value >= (uint64_t)s->E * s->A * s->K) return fail(PIC_ERR_INVALID_ARG, "first view out of range");
            s->view_first = (long long)value; return PIC_OK;
        case PIC_OPT_VIEW_COUNT: s->view_count = (long long)value; return PIC_OK;
        case PIC_OPT_DEBUG_FLAGS: s->debug_flags = (int)value; return PIC_OK;
        case PIC_OPT_OUT_RELATIVE: s->out_relative = value != 0; return PIC_OK;
        case PIC_OPT_TIMING: {
            if (value && !s->ev) {
                DeviceGuard guard(s->device);
                if (!guard.ok) return fail(PIC_ERR_CUDA, "cannot select device %d", s->device);
                s->ev = new (std::nothrow) cudaEvent_t[2 * kMaxTimed]();
                if (!s->ev) return fail(PIC_ERR_OOM, "host allocation failed");
                for (int i = 0; i < 2 * kMaxTimed; ++i) CUDA_TRY(cudaEventCreate(&s->ev[i]));
            }
            s->timing = value != 0;
            s->n_timed = 0;
            return PIC_OK;
        }
        default: return fail(PIC_ERR_INVALID_ARG, "unknown option %d", option);
    }
}

static pic_status render_from(pic_scene* s, const float* poses, float* state, const float* actions, const float* dims,
                              const uint8_t* active, const pic_camera* rig, uint8_t* out_class, uint16_t* out_depth,
                              cudaStream_t stream, uint8_t* out_rgb = nullptr, bool antialias = false) {
    pic::RenderParams P;
    pic_status st = fill_params(s, rig, out_class, out_depth, P, out_rgb != nullptr);
    if (st != PIC_OK) return st;
    P.out_rgb = out_rgb;
    DeviceGuard guard(s->device);
    if (!guard.ok) return fail(PIC_ERR_CUDA, "cannot select device %d", s->device);
    const int n_agents = s->E * s->A;
    CUDA_TRY(pic::launch_setup(P, n_agents, poses, state, actions, dims, active, s->have_agent_cls ? s->d_agent_cls : nullptr, s->d_agents, s->d_cams, s->d_tables,
                               s->d_status, kDt, kWheelbase, kVMax, stream));
    const long long total = (long long)s->E * s->A * s->K;
    long long count = total - s->view_first;
    if (s->view_count > 0 && s->view_count < count) count = s->view_count;
    P.view_first = s->view_first;
    if (s->out_relative) {
        // the caller's buffers start at the first rendered view: shift the bases so that the kernels'
        // absolute view indexing lands there (never dereferenced below view_first)
        const size_t off = (size_t)s->view_first * s->H * s->W;
        if (P.out_class) { P.out_class -= off; P.out_depth -= off; }
        if (P.out_depth32) P.out_depth32 -= off;
        if (P.out_rgb) P.out_rgb -= 3 * off;
    }
    if (out_rgb) P.occlusion = nullptr;
    if (P.occlusion)    // the counts of the rendered views start at zero
        CUDA_TRY(cudaMemsetAsync(P.occlusion + (size_t)s->view_first * s->A * 2, 0, sizeof(uint32_t) * 2 * (size_t)count * s->A, stream));
    const bool timed = s->timing && s->n_timed < kMaxTimed;
    if (timed) CUDA_TRY(cudaEventRecord(s->ev[2 * s->n_timed], stream));
    if (out_rgb) CUDA_TRY(pic::launch_colour(P, count, antialias, stream));
    else CUDA_TRY(pic::launch_render(P, count, s->brute, s->sm_count, stream));
    if (timed) { CUDA_TRY(cudaEventRecord(s->ev[2 * s->n_timed + 1], stream)); ++s->n_timed; }
    return PIC_OK;
}

pic_status pic_render(pic_scene* s, const float* poses, const float* dims, const uint8_t* active, const pic_camera* rig,
                      uint8_t* out_class, uint16_t* out_depth, void* cuda_stream) {
    if (!s) return fail(PIC_ERR_INVALID_ARG, "scene is NULL");
    if (!poses || !dims) return fail(PIC_ERR_INVALID_ARG, "poses or dims is NULL");
    return render_from(s, poses, nullptr, nullptr, dims, active, rig, out_class, out_depth, static_cast<cudaStream_t>(cuda_stream));
}

pic_status pic_set_palette(pic_scene* s, const uint8_t* rgb, void* cuda_stream) {
    if (!s || !rgb) return fail(PIC_ERR_INVALID_ARG, "scene or palette is NULL");
    DeviceGuard guard(s->device);
    if (!guard.ok) return fail(PIC_ERR_CUDA, "cannot select device %d", s->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    CUDA_TRY(cudaMemcpyAsync(s->d_palette, rgb, 768, cudaMemcpyHostToDevice, stream));
    CUDA_TRY(cudaStreamSynchronize(stream));          // the host array may be reused by the caller
    return PIC_OK;
}

pic_status pic_render_rgb(pic_scene* s, const float* poses, const float* dims, const uint8_t* active, const pic_camera* rig,
                          int32_t antialias, uint8_t* out_rgb, void* cuda_stream) {
    if (!s) return fail(PIC_ERR_INVALID_ARG, "scene is NULL");
    if (!poses || !dims || !out_rgb) return fail(PIC_ERR_INVALID_ARG, "poses, dims or out_rgb is NULL");
    return render_from(s, poses, nullptr, nullptr, dims, active, rig, nullptr, nullptr, static_cast<cudaStream_t>(cuda_stream), out_rgb,
                       antialias != 0);
}

pic_status pic_render_host(pic_scene* s, const float* poses, const float* dims, const uint8_t* active,
                           const pic_camera* rig, uint8_t* out_class, uint16_t* out_depth, void* cuda_stream) {
    if (!s) return fail(PIC_ERR_INVALID_ARG, "scene is NULL");
    if (!poses || !dims || !out_class || !out_depth) return fail(PIC_ERR_INVALID_ARG, "a required host pointer is NULL");
    DeviceGuard guard(s->device);
    if (!guard.ok) return fail(PIC_ERR_CUDA, "cannot select device %d", s->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t n_agents = (size_t)s->E * s->A;
    const size_t n_px = n_agents * s->K * s->H * s->W;
    if (!s->d_out_class) {
        CUDA_TRY(cudaMalloc((void**)&s->d_in_poses, sizeof(float) * 3 * n_agents));
        CUDA_TRY(cudaMalloc((void**)&s->d_in_dims, sizeof(float) * 3 * n_agents));
        CUDA_TRY(cudaMalloc((void**)&s->d_in_active, n_agents));
        CUDA_TRY(cudaMalloc((void**)&s->d_out_depth, sizeof(uint16_t) * n_px));
        CUDA_TRY(cudaMalloc((void**)&s->d_out_class, n_px));
    }
    CUDA_TRY(cudaMemcpyAsync(s->d_in_poses, poses, sizeof(float) * 3 * n_agents, cudaMemcpyHostToDevice, stream));
    CUDA_TRY(cudaMemcpyAsync(s->d_in_dims, dims, sizeof(float) * 3 * n_agents, cudaMemcpyHostToDevice, stream));
    if (active) CUDA_TRY(cudaMemcpyAsync(s->d_in_active, active, n_agents, cudaMemcpyHostToDevice, stream));
    pic_status st = render_from(s, s->d_in_poses, nullptr, nullptr, s->d_in_dims, active ? s->d_in_active : nullptr, rig,
                                s->d_out_class, s->d_out_depth, stream);
    if (st != PIC_OK) return st;
    CUDA_TRY(cudaMemcpyAsync(out_class, s->d_out_class, n_px, cudaMemcpyDeviceToHost, stream));
    CUDA_TRY(cudaMemcpyAsync(out_depth, s->d_out_depth, sizeof(uint16_t) * n_px, cudaMemcpyDeviceToHost, stream));
    CUDA_TRY(cudaStreamSynchronize(stream));
    return PIC_OK;
}

pic_status pic_set_state(pic_scene* s, const float* state, const float* dims, const uint8_t* active, void* cuda_stream) {
    if (!s) return fail(PIC_ERR_INVALID_ARG, "scene is NULL");
    if (!state || !dims) return fail(PIC_ERR_INVALID_ARG, "state or dims is NULL");
    DeviceGuard guard(s->device);
    if (!guard.ok) return fail(PIC_ERR_CUDA, "cannot select device %d", s->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t n = (size_t)s->E * s->A;
    CUDA_TRY(cudaMemcpyAsync(s->d_state, state, sizeof(float) * 4 * n, cudaMemcpyDeviceToDevice, stream));
    CUDA_TRY(cudaMemcpyAsync(s->d_dims, dims, sizeof(float) * 3 * n, cudaMemcpyDeviceToDevice, stream));
    if (active) CUDA_TRY(cudaMemcpyAsync(s->d_active, active, n, cudaMemcpyDeviceToDevice, stream));
    else CUDA_TRY(cudaMemsetAsync(s->d_active, 1, n, stream));
    return PIC_OK;
}

pic_status pic_set_agent_classes(pic_scene* s, const uint8_t* classes, void* cuda_stream) {
    if (!s) return fail(PIC_ERR_INVALID_ARG, "scene is NULL");
    DeviceGuard guard(s->device);
    if (!guard.ok) return fail(PIC_ERR_CUDA, "cannot select device %d", s->device);
    s->have_agent_cls = classes != nullptr;
    if (classes)
        CUDA_TRY(cudaMemcpyAsync(s->d_agent_cls, classes, (size_t)s->E * s->A, cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(cuda_stream)));
    return PIC_OK;
}

pic_status pic_get_state(pic_scene* s, float* state_out, void* cuda_stream) {
    if (!s) return fail(PIC_ERR_INVALID_ARG, "scene is NULL");
    if (!state_out) return fail(PIC_ERR_INVALID_ARG, "state_out is NULL");
    DeviceGuard guard(s->device);
    if (!guard.ok) return fail(PIC_ERR_CUDA, "cannot select device %d", s->device);
    const size_t n = (size_t)s->E * s->A;
    CUDA_TRY(cudaMemcpyAsync(state_out, s->d_state, sizeof(float) * 4 * n, cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(cuda_stream)));
    return PIC_OK;
}

pic_status pic_step(pic_scene* s, const float* actions, const pic_camera* rig, uint8_t* out_class, uint16_t* out_depth,
                    void* cuda_stream) {
    if (!s) return fail(PIC_ERR_INVALID_ARG, "scene is NULL");
    if (!actions) return fail(PIC_ERR_INVALID_ARG, "actions is NULL");
    return render_from(s, nullptr, s->d_state, actions, s->d_dims, s->d_active, rig, out_class, out_depth,
                       static_cast<cudaStream_t>(cuda_stream));
}

pic_status pic_step_rgb(pic_scene* s, const float* actions, const pic_camera* rig, int32_t antialias, uint8_t* out_rgb,
                        void* cuda_stream) {
    if (!s) return fail(PIC_ERR_INVALID_ARG, "scene is NULL");
    if (!actions || !out_rgb) return fail(PIC_ERR_INVALID_ARG, "actions or out_rgb is NULL");
    return render_from(s, nullptr, s->d_state, actions, s->d_dims, s->d_active, rig, nullptr, nullptr,
                       static_cast<cudaStream_t>(cuda_stream), out_rgb, antialias != 0);
}

pic_status pic_get_kernel_times(pic_scene* s, float* ms, int32_t capacity, int32_t* n) {
    if (!s) return fail(PIC_ERR_INVALID_ARG, "scene is NULL");
    if (!n || (capacity > 0 && !ms)) return fail(PIC_ERR_INVALID_ARG, "ms or n is NULL");
    DeviceGuard guard(s->device);
    if (!guard.ok) return fail(PIC_ERR_CUDA, "cannot select device %d", s->device);
    *n = s->n_timed;
    for (int i = 0; i < s->n_timed; ++i) {
        CUDA_TRY(cudaEventSynchronize(s->ev[2 * i + 1]));
        if (i < capacity) CUDA_TRY(cudaEventElapsedTime(&ms[i], s->ev[2 * i], s->ev[2 * i + 1]));
    }
    s->n_timed = 0;
    return PIC_OK;
}

pic_status pic_get_status(pic_scene* s, uint32_t* flags, void* cuda_stream) {
    if (!s) return fail(PIC_ERR_INVALID_ARG, "scene is NULL");
    if (!flags) return fail(PIC_ERR_INVALID_ARG, "flags is NULL");
    DeviceGuard guard(s->device);
    if (!guard.ok) return fail(PIC_ERR_CUDA, "cannot select device %d", s->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    CUDA_TRY(cudaMemcpyAsync(flags, s->d_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, stream));
    CUDA_TRY(cudaMemsetAsync(s->d_status, 0, sizeof(uint32_t), stream));
    CUDA_TRY(cudaStreamSynchronize(stream));
    return PIC_OK;
}

}  // extern "C"
