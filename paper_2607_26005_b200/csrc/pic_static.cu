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
#include "pic_exhaustive.cuh"

namespace pic {
cudaError_t launch_setup(const RenderParams& P, int n_agents, const float* poses, float* state, const float* actions,
                         const float* dims, const uint8_t* active, const uint8_t* agent_cls, AgentGeom* agents_out, ViewCam* cams_out,
                         float* tables, uint32_t* status, float dt, float wheelbase, float v_max, cudaStream_t stream);
void set_last_error(const char* msg);
}  // namespace pic

namespace {

using namespace pic;

constexpr int kMaxAgents = PIC_STATIC_MAX_AGENTS;
constexpr int kMaxViews = PIC_STATIC_MAX_VIEWS;
constexpr int kMaxSide = PIC_STATIC_MAX_SIDE;
constexpr int kMaxDevices = 64;

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

__device__ __forceinline__ bool lex_less(float ax, float ay, float az, float bx, float by, float bz) {
    if (ax != bx) return ax < bx;
    if (ay != by) return ay < by;
    return az < bz;
}

// The exhaustive tile renderer over the caller's raw triangles.
__global__ void __launch_bounds__(EXH_THREADS) render_static_kernel(const __grid_constant__ StaticParams S) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    ExhaustiveSmem& s = *reinterpret_cast<ExhaustiveSmem*>(smem_raw);
    const float* tri_xyz = S.tri_xyz;
    const uint8_t* tri_class = S.tri_class;
    exhaustive_tile(s, S.P, blockIdx.x, S.n_tris, S.n_tris,
                    [tri_xyz, tri_class](uint32_t i, const Cam& c, V3 (&V)[4], V3& Pn, bool& quad, uint32_t& flags, uint32_t& key_lo) {
                        const float* p = tri_xyz + 9 * (size_t)i;
                        float v[9];
#pragma unroll
                        for (int j = 0; j < 9; ++j) v[j] = __ldg(p + j);
#pragma unroll
                        for (int j = 0; j < 3; ++j) V[j] = to_camera(c, v[3 * j], v[3 * j + 1], v[3 * j + 2]);
                        V[3] = V[2];
                        const float v12[12] = {v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7], v[8], v[6], v[7], v[8]};
                        Pn = plane_normal_world(c, v12, false);
                        quad = false;
                        flags = 0u;
                        // an edge shared by two triangles is evaluated in the same direction by both
                        if (!lex_less(v[0], v[1], v[2], v[3], v[4], v[5])) flags |= 1u << 4;
                        if (!lex_less(v[3], v[4], v[5], v[6], v[7], v[8])) flags |= 1u << 5;
                        if (!lex_less(v[6], v[7], v[8], v[0], v[1], v[2])) flags |= 1u << 6;
                        key_lo = ((0xFFFFFFu - i) << 8) | __ldg(tri_class + i);
                    });
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
    {
        // every primitive is tested against every pixel of every view: bound the product, so that a
        // request at all the limits at once cannot occupy the GPU for hours
        const double work = ((double)d->n_tris + 6.0 * d->A) * (double)d->E * d->A * d->K * (double)d->H * d->W;
        if (work > (double)PIC_STATIC_MAX_WORK)
            return fail(PIC_ERR_CAPACITY, "pic_render_static: (n_tris + 6A) * E*A*K*H*W = %.3g primitive-pixel tests, at most %.3g", work,
                        (double)PIC_STATIC_MAX_WORK);
    }
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
            ce = cudaFuncSetAttribute(render_static_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ExhaustiveSmem));
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
    // (the status word is sticky across calls, like a scene's: pic_static_status reads and clears it)
    ce = pic::launch_setup(P, d->E * d->A, poses, nullptr, nullptr, dims, active, nullptr, agents, cams, tables, status, 0.f, 1.f, 0.f, stream);
    if (ce != cudaSuccess) return fail(PIC_ERR_CUDA, "set-up kernels: %s", cudaGetErrorString(ce));
    const unsigned blocks = (unsigned)(d->E * d->A * d->K * P.tiles_x * P.tiles_y);
    render_static_kernel<<<blocks, EXH_THREADS, sizeof(ExhaustiveSmem), stream>>>(S);
    ce = cudaGetLastError();
    if (ce != cudaSuccess) return fail(PIC_ERR_CUDA, "render_static_kernel: %s", cudaGetErrorString(ce));
    return PIC_OK;
}

extern "C" pic_status pic_static_status(uint32_t* flags, void* cuda_stream) {
    if (!flags) return fail(PIC_ERR_INVALID_ARG, "flags is NULL");
    *flags = 0u;
    int dev = -1;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce != cudaSuccess) return fail(PIC_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(ce));
    if (dev < 0 || dev >= kMaxDevices) return fail(PIC_ERR_INVALID_ARG, "device ordinal %d not supported", dev);
    unsigned char* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        scratch = g_scratch_ptr[dev];
    }
    if (!scratch) return PIC_OK;                  // pic_render_static has not run on this device
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint32_t* status = reinterpret_cast<uint32_t*>(scratch + kOffStatus);
    ce = cudaMemcpyAsync(flags, status, sizeof(uint32_t), cudaMemcpyDeviceToHost, stream);
    if (ce == cudaSuccess) ce = cudaMemsetAsync(status, 0, sizeof(uint32_t), stream);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(stream);
    if (ce != cudaSuccess) return fail(PIC_ERR_CUDA, "reading the status word: %s", cudaGetErrorString(ce));
    return PIC_OK;
}
