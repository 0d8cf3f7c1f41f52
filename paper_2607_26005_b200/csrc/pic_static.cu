// pic_render_static: a self-contained render call for hosts that must not allocate device memory.
//
// Everything the ordinary path keeps in buffers obtained with cudaMalloc when a scene is created --
// per-agent geometry, per-view cameras, per-camera ray/background tables, the status word -- lives
// here in ONE file-scope device array of fixed size.  The map is read straight from the caller's
// triangle arrays (no hierarchy is built), so the call needs no scene object at all.
//
// In host code the name of a __device__ array is only a stand-in for the symbol, not an address a
// kernel can use; its device address is looked up with cudaGetSymbolAddress, once per device,
// with that device current, and handed to the kernels as an ordinary pointer.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "../../include/pictura.h"
#include "pic_device.cuh"

namespace pic {
cudaError_t launch_setup(const RenderParams& P, int n_agents, const float* poses, float* state, const float* actions,
                         const float* dims, const uint8_t* active, AgentGeom* agents_out, ViewCam* cams_out,
                         float* tables, uint32_t* status, float dt, float wheelbase, float v_max, cudaStream_t stream);
void set_last_error(const char* msg);
}  // namespace pic

namespace {

using namespace pic;

constexpr int kMaxAgents = PIC_STATIC_MAX_AGENTS;
constexpr int kMaxViews = PIC_STATIC_MAX_VIEWS;
constexpr int kMaxSide = PIC_STATIC_MAX_SIDE;
constexpr int kMaxDevices = 64;
constexpr int kThreads = 128;

// scratch layout (bytes)
constexpr size_t kOffAgents = 0;
constexpr size_t kOffCams = kOffAgents + sizeof(AgentGeom) * kMaxAgents;
constexpr size_t kOffTables = kOffCams + sizeof(ViewCam) * kMaxViews;
constexpr size_t kOffStatus = kOffTables + sizeof(float) * MAX_CAMS * 4 * kMaxSide;
constexpr size_t kScratchBytes = kOffStatus + 256;

// The only device memory this entry point ever uses besides the caller's buffers (about 420 KB,
// held by every device that loads the library until the process exits).
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

std::mutex g_mutex;
unsigned char* g_scratch_ptr[kMaxDevices] = {};     // device address of g_static_scratch, per device

struct StaticParams {
    RenderParams P;
    const float* tri_xyz;        // dev [N,3,3]
    const uint8_t* tri_class;    // dev [N]
    uint32_t n_tris;
};

struct __align__(16) StaticSmem {
    unsigned long long key[TILE * TILE];
    float ray_x[TILE], ray_y[TILE];
    Cam cam;
};

__device__ __forceinline__ bool lex_less(float ax, float ay, float az, float bx, float by, float bz) {
    if (ax != bx) return ax < bx;
    if (ay != by) return ay < by;
    return az < bz;
}

// Variant of the exhaustive kernel that reads the caller's raw triangles: every triangle and every
// face of every other agent's box against every pixel of a 64 x 64 tile.
__global__ void __launch_bounds__(kThreads) render_static_kernel(const __grid_constant__ StaticParams S) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    StaticSmem& s = *reinterpret_cast<StaticSmem*>(smem_raw);
    const RenderParams& P = S.P;
    const unsigned tiles = (unsigned)(P.tiles_x * P.tiles_y);
    const unsigned job = blockIdx.x;
    const unsigned view = job / tiles;
    const int tile = (int)(job % tiles);
    const int k = (int)(view % (unsigned)P.K);
    const int a = (int)((view / (unsigned)P.K) % (unsigned)P.A);
    const int e = (int)(view / ((unsigned)P.K * (unsigned)P.A));
    TileCtx t;
    t.x0 = (tile % P.tiles_x) * TILE; t.y0 = (tile / P.tiles_x) * TILE;
    t.tw = min(TILE, P.W - t.x0); t.th = min(TILE, P.H - t.y0);
    t.w_near = P.w_near; t.w_far = P.w_far; t.near_z = P.near_z; t.far_z = P.far_z;
    const AgentGeom ego = P.agents[(size_t)e * P.A + a];
    if (threadIdx.x == 0) load_camera(s.cam, P.cams[view], P.cam[k], P.W, P.H);
    for (int i = threadIdx.x; i < TILE * TILE; i += kThreads) s.key[i] = 0ull;
    if (threadIdx.x < TILE) {
        const int i = threadIdx.x;
        s.ray_x[i] = (t.x0 + i < P.W) ? P.rig.ray_x[(size_t)k * P.W + t.x0 + i] : 0.f;
        s.ray_y[i] = (t.y0 + i < P.H) ? P.rig.ray_y[(size_t)k * P.H + t.y0 + i] : 0.f;
    }
    __syncthreads();
    const Cam& c = s.cam;
    if (ego.active) {
        const uint32_t n_items = S.n_tris + 6u * (uint32_t)P.A;
        for (uint32_t i = threadIdx.x; i < n_items; i += kThreads) {
            V3 V[4], Pn; bool quad; uint32_t flags, key_lo;
            if (i < S.n_tris) {
                const float* p = S.tri_xyz + 9 * (size_t)i;
                float v[9];
#pragma unroll
                for (int j = 0; j < 9; ++j) v[j] = __ldg(p + j);
#pragma unroll
                for (int j = 0; j < 3; ++j) V[j] = to_camera(c, v[3 * j], v[3 * j + 1], v[3 * j + 2]);
                V[3] = V[2];
                {
                    const float v12[12] = {v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7], v[8], v[6], v[7], v[8]};
                    Pn = plane_normal_world(c, v12, false);
                }
                quad = false;
                flags = 0u;
                // an edge shared by two triangles is evaluated in the same direction by both
                if (!lex_less(v[0], v[1], v[2], v[3], v[4], v[5])) flags |= 1u << 4;
                if (!lex_less(v[3], v[4], v[5], v[6], v[7], v[8])) flags |= 1u << 5;
                if (!lex_less(v[6], v[7], v[8], v[0], v[1], v[2])) flags |= 1u << 6;
                key_lo = ((0xFFFFFFu - i) << 8) | __ldg(S.tri_class + i);
            } else {
                const uint32_t j = i - S.n_tris;
                const int b = (int)(j / 6u), f = (int)(j % 6u);
                if (b == a) continue;
                const AgentGeom g = P.agents[(size_t)e * P.A + b];
                if (!g.active) continue;
                const uint32_t corners = face_corners(f);
#pragma unroll
                for (int q = 0; q < 4; ++q) V[q] = box_corner(c, g, (corners >> (4 * q)) & 7u);
                quad = true; flags = face_flags(corners);
                key_lo = ((0xFFFFFFu - (S.n_tris + 12u * (uint32_t)b + 2u * (uint32_t)f)) << 8) | P.cls_agent;
                Pn = plane_normal(V, true);
            }
            PrimEq q;
            if (!prim_equations(V, quad, flags, Pn, q)) continue;
            for (int y = 0; y < t.th; ++y) {
                const float ry = s.ray_y[y];
                for (int x = 0; x < t.tw; ++x) {
                    const uint32_t wb = fragment(q, s.ray_x[x], ry, t.w_near, t.w_far);
                    if (wb) {
                        const unsigned long long key = make_key(wb, key_lo);
                        unsigned long long* addr = &s.key[y * TILE + x];
                        if (key > *reinterpret_cast<volatile unsigned long long*>(addr)) atomicMax(addr, key);
                    }
                }
            }
        }
    }
    __syncthreads();
    const size_t img = (size_t)P.H * P.W;
    uint8_t* oc = P.out_class + view * img;
    uint16_t* od = P.out_depth + view * img;
    for (int i = threadIdx.x; i < t.th * t.tw; i += kThreads) {
        const int y = i / t.tw, x = i % t.tw;
        uint32_t cls = P.cls_sky; float z = P.far_z;
        if (ego.active) { cls = P.rig.bg_cls[(size_t)k * P.H + t.y0 + y]; z = P.rig.bg_z[(size_t)k * P.H + t.y0 + y]; }
        const unsigned long long key = s.key[y * TILE + x];
        if (key) { cls = (uint32_t)(key & 0xff); z = fast_rcp(__uint_as_float((uint32_t)(key >> 32))); }
        const size_t o = (size_t)(t.y0 + y) * P.W + t.x0 + x;
        oc[o] = (uint8_t)cls;
        od[o] = __half_as_ushort(__float2half_rn(z));
    }
}

pic_status fail(pic_status st, const char* fmt, ...) {
    char buf[384];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    pic::set_last_error(buf);
    return st;
}

}  // namespace

extern "C" pic_status pic_render_static(const pic_static_desc* d, const float* tri_xyz, const uint8_t* tri_class,
                                        const float* poses, const float* dims, const uint8_t* active,
                                        const pic_camera* rig, uint8_t* out_class, uint16_t* out_depth, void* cuda_stream) {
    if (!d) return fail(PIC_ERR_INVALID_ARG, "desc is NULL");
    if (d->size != sizeof(pic_static_desc)) return fail(PIC_ERR_INVALID_ARG, "desc->size is %u, expected %zu", d->size, sizeof(pic_static_desc));
    if (d->E <= 0 || d->A <= 0 || d->K <= 0 || d->H <= 0 || d->W <= 0 || d->n_tris < 0) return fail(PIC_ERR_SHAPE, "sizes must be positive");
    if (d->K > MAX_CAMS) return fail(PIC_ERR_SHAPE, "at most %d cameras per rig", MAX_CAMS);
    if ((long long)d->E * d->A > kMaxAgents)
        return fail(PIC_ERR_CAPACITY, "pic_render_static holds at most %d agents (E*A), got %lld", kMaxAgents, (long long)d->E * d->A);
    if ((long long)d->E * d->A * d->K > kMaxViews)
        return fail(PIC_ERR_CAPACITY, "pic_render_static holds at most %d views (E*A*K), got %lld", kMaxViews, (long long)d->E * d->A * d->K);
    if (d->H > kMaxSide || d->W > kMaxSide)
        return fail(PIC_ERR_CAPACITY, "pic_render_static renders images up to %d x %d, got %d x %d", kMaxSide, kMaxSide, d->H, d->W);
    if (d->n_tris > PIC_STATIC_MAX_TRIS) return fail(PIC_ERR_CAPACITY, "pic_render_static reads at most %d triangles, got %d", PIC_STATIC_MAX_TRIS, d->n_tris);
    if (!(d->near_z > 0.f) || !(d->far_z > d->near_z) || !std::isfinite(d->far_z)) return fail(PIC_ERR_INVALID_ARG, "need 0 < near_z < far_z < inf");
    if (!poses || !dims || !rig || !out_class || !out_depth) return fail(PIC_ERR_INVALID_ARG, "a required pointer is NULL");
    if (d->n_tris > 0 && (!tri_xyz || !tri_class)) return fail(PIC_ERR_INVALID_ARG, "triangle arrays are NULL");
    for (int k = 0; k < d->K; ++k) {
        const float vals[7] = {rig[k].mount_x, rig[k].mount_y, rig[k].mount_z, rig[k].yaw, rig[k].pitch, rig[k].fx, rig[k].fy};
        for (float v : vals)
            if (!std::isfinite(v)) return fail(PIC_ERR_INVALID_ARG, "camera %d has a non-finite field", k);
        if (!(rig[k].fx > 0.f) || !(rig[k].fy > 0.f)) return fail(PIC_ERR_INVALID_ARG, "camera %d: focal lengths must be positive", k);
    }
    int dev = -1;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce != cudaSuccess) return fail(PIC_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(ce));
    if (dev < 0 || dev >= kMaxDevices) return fail(PIC_ERR_INVALID_ARG, "device ordinal %d not supported", dev);
    unsigned char* scratch = nullptr;
    {
        // once per device, with that device current: the device address of the static array
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!g_scratch_ptr[dev]) {
            void* p = nullptr;
            ce = cudaGetSymbolAddress(&p, g_static_scratch);
            if (ce != cudaSuccess) return fail(PIC_ERR_CUDA, "cudaGetSymbolAddress: %s", cudaGetErrorString(ce));
            ce = cudaFuncSetAttribute(render_static_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(StaticSmem));
            if (ce != cudaSuccess) return fail(PIC_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(ce));
            g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
        }
        scratch = g_scratch_ptr[dev];
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    StaticParams S;
    memset(&S, 0, sizeof(S));
    RenderParams& P = S.P;
    P.E = d->E; P.A = d->A; P.K = d->K; P.H = d->H; P.W = d->W;
    P.tiles_x = (d->W + TILE - 1) / TILE; P.tiles_y = (d->H + TILE - 1) / TILE;
    P.near_z = d->near_z; P.far_z = d->far_z; P.w_near = 1.0f / d->near_z; P.w_far = 1.0f / d->far_z;
    P.cls_agent = d->agent_class; P.cls_sky = d->sky_class; P.cls_ground = d->ground_class;
    AgentGeom* agents = reinterpret_cast<AgentGeom*>(scratch + kOffAgents);
    ViewCam* cams = reinterpret_cast<ViewCam*>(scratch + kOffCams);
    float* tables = reinterpret_cast<float*>(scratch + kOffTables);
    uint32_t* status = reinterpret_cast<uint32_t*>(scratch + kOffStatus);
    P.agents = agents; P.cams = cams;
    P.rig.ray_x = tables;
    P.rig.ray_y = P.rig.ray_x + (size_t)d->K * d->W;
    P.rig.bg_z = P.rig.ray_y + (size_t)d->K * d->H;
    P.rig.bg_cls = reinterpret_cast<const uint32_t*>(P.rig.bg_z + (size_t)d->K * d->H);
    P.out_class = out_class; P.out_depth = out_depth;
    for (int k = 0; k < d->K; ++k) {
        CamConst& o = P.cam[k];
        o.mx = rig[k].mount_x; o.my = rig[k].mount_y; o.mz = rig[k].mount_z;
        o.cpsi = (float)std::cos((double)rig[k].yaw); o.spsi = (float)std::sin((double)rig[k].yaw);
        o.cphi = (float)std::cos((double)rig[k].pitch); o.sphi = (float)std::sin((double)rig[k].pitch);
        o.fx = rig[k].fx; o.fy = rig[k].fy;
    }
    S.tri_xyz = tri_xyz; S.tri_class = tri_class; S.n_tris = (uint32_t)d->n_tris;
    // the array keeps whatever the previous call left: the status word must start at zero
    ce = cudaMemsetAsync(status, 0, sizeof(uint32_t), stream);
    if (ce != cudaSuccess) return fail(PIC_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(ce));
    ce = pic::launch_setup(P, d->E * d->A, poses, nullptr, nullptr, dims, active, agents, cams, tables, status, 0.f, 1.f, 0.f, stream);
    if (ce != cudaSuccess) return fail(PIC_ERR_CUDA, "set-up kernels: %s", cudaGetErrorString(ce));
    const unsigned blocks = (unsigned)(d->E * d->A * d->K * P.tiles_x * P.tiles_y);
    render_static_kernel<<<blocks, kThreads, sizeof(StaticSmem), stream>>>(S);
    ce = cudaGetLastError();
    if (ce != cudaSuccess) return fail(PIC_ERR_CUDA, "render_static_kernel: %s", cudaGetErrorString(ce));
    return PIC_OK;
}
