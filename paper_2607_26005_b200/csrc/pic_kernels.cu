// Agent kernel, rig-table kernel, exhaustive cross-check kernel and host-side launchers.
//
// The exhaustive kernel (see pic_exhaustive.cuh) is the cross-check of the production kernels in
// pic_render.cu.
#include "pic_exhaustive.cuh"

namespace pic {

struct RigParams {
    int32_t K, W, H;
    float far_z;
    uint32_t cls_sky, cls_ground;
    CamConst cam[MAX_CAMS];
};

// ------------------------------------------------------------------------------------------------
// agent kernel: poses/dims/active -> AgentGeom + one ViewCam per camera (optionally after one
// kinematic-bicycle step of the scene's own state)
// ------------------------------------------------------------------------------------------------
__global__ void agent_kernel(int n, const float* __restrict__ poses, float* state, const float* __restrict__ actions,
                             const float* __restrict__ dims, const uint8_t* __restrict__ active,
                             const uint8_t* __restrict__ agent_cls, uint32_t default_cls, AgentGeom* __restrict__ out, ViewCam* __restrict__ cams, uint32_t* status,
                             const __grid_constant__ RigParams R, float dt, float wheelbase, float v_max) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    bool act = active ? active[i] != 0 : true;
    float x, y, th;
    if (state) {                                   // pic_step: update the scene's own state in place
        float v;
        x = state[4 * i]; y = state[4 * i + 1]; th = state[4 * i + 2]; v = state[4 * i + 3];
        if (actions && act) {
            const float acc = actions[2 * i], steer = actions[2 * i + 1];
            float s, c;
            sincosf(th, &s, &c);
            const float nx = fm(mul(v, c), dt, x);
            const float ny = fm(mul(v, s), dt, y);
            const float nth = fm(mul(__fdiv_rn(v, wheelbase), tanf(steer)), dt, th);
            const float nv = fminf(fmaxf(fm(acc, dt, v), 0.f), v_max);
            if (isfinite(acc) && isfinite(steer) && isfinite(nx) && isfinite(ny) && isfinite(nth) && isfinite(nv)) {
                x = nx; y = ny; th = nth; v = nv;
                state[4 * i] = x; state[4 * i + 1] = y; state[4 * i + 2] = th; state[4 * i + 3] = v;
            } else {
                // a non-finite action (or a step that overflows) is flagged, leaves the agent's
                // state as it was and takes the agent out of this step's images
                atomicOr(status, 1u);
                act = false;
            }
        }
    } else {
        x = poses[3 * i]; y = poses[3 * i + 1]; th = poses[3 * i + 2];
    }
    float l = dims[3 * i], w = dims[3 * i + 1], h = dims[3 * i + 2];
    if (!(isfinite(x) && isfinite(y) && isfinite(th) && isfinite(l) && isfinite(w) && isfinite(h))) {
        atomicOr(status, 1u);
        act = false;
        x = y = th = 0.f; l = w = h = 1.f;
    }
    AgentGeom g;
    g.x = x; g.y = y;
    sincosf(th, &g.s, &g.c);
    g.hl = 0.5f * l; g.hw = 0.5f * w; g.h = h;
    g.active = act ? (1u | ((agent_cls ? (uint32_t)agent_cls[i] : default_cls) << 8)) : 0u;
    out[i] = g;
    for (int k = 0; k < R.K; ++k) {
        ViewCam vc;
        make_view_cam(vc, g, R.cam[k]);
        float4* dst = reinterpret_cast<float4*>(cams + (size_t)i * R.K + k);
        const float4* src = reinterpret_cast<const float4*>(&vc);
        dst[0] = src[0]; dst[1] = src[1]; dst[2] = src[2]; dst[3] = src[3];
    }
}

// Per-camera tables: ray coordinates of every pixel column / row and the background of every row.
__global__ void rig_kernel(const __grid_constant__ RigParams R, float* __restrict__ ray_x, float* __restrict__ ray_y,
                           float* __restrict__ bg_z, uint32_t* __restrict__ bg_cls, uint32_t* overflow) {
    const int k = blockIdx.x;
    if (overflow && k == 0 && threadIdx.x == 0) overflow[0] = 0u;   // the render kernels' list of left-out tiles starts empty (absent for callers that do not use them)
    const CamConst c = R.cam[k];
    const float cx = 0.5f * (float)R.W, cy = 0.5f * (float)R.H;
    for (int u = threadIdx.x; u < R.W; u += blockDim.x)
        ray_x[(size_t)k * R.W + u] = __fdiv_rn(sub(add((float)u, 0.5f), cx), c.fx);
    for (int v = threadIdx.x; v < R.H; v += blockDim.x) {
        const float ry = __fdiv_rn(sub(add((float)v, 0.5f), cy), c.fy);
        ray_y[(size_t)k * R.H + v] = ry;
        uint32_t cls; float z;
        background(c.cphi, c.sphi, c.mz, ry, R.far_z, R.cls_sky, R.cls_ground, cls, z);
        bg_z[(size_t)k * R.H + v] = z;
        bg_cls[(size_t)k * R.H + v] = cls;
    }
}

// ------------------------------------------------------------------------------------------------
// exhaustive kernel: the scene's preprocessed primitives through the shared exhaustive tile renderer
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(EXH_THREADS) render_brute_kernel(const __grid_constant__ RenderParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    ExhaustiveSmem& s = *reinterpret_cast<ExhaustiveSmem*>(smem_raw);
    const unsigned tiles = (unsigned)(P.tiles_x * P.tiles_y);
    const int e = (int)(((size_t)P.view_first + blockIdx.x / tiles) / ((size_t)P.K * P.A));
    const MapInfo mi = P.maps[P.env_map[e]];
    const Prim* prims = P.prims + mi.prim_begin;
    exhaustive_tile(s, P, blockIdx.x, mi.prim_end - mi.prim_begin, mi.n_tris,
                    [prims](uint32_t i, const Cam& c, V3 (&V)[4], V3& Pn, bool& quad, uint32_t& flags, uint32_t& key_lo) {
                        float v[12], vis_cos;
                        load_prim(prims + i, v, key_lo, flags, vis_cos);
                        quad = flags & 1u;
#pragma unroll
                        for (int j = 0; j < 4; ++j) V[j] = to_camera(c, v[3 * j], v[3 * j + 1], v[3 * j + 2]);
                        Pn = limit_angular_range(V, plane_normal_world(c, v, quad), vis_cos);
                    });
}

// ------------------------------------------------------------------------------------------------
// host-side launchers (called from the C ABI)
// ------------------------------------------------------------------------------------------------
size_t render_smem_bytes();                       // pic_render.cu
cudaError_t configure_render_kernel();            // pic_render.cu
cudaError_t launch_render_kernel(const RenderParams& P, long long n_views, int sm_count, cudaStream_t stream);
cudaError_t launch_coverage_kernel(const RenderParams& P, long long n_views, cudaStream_t stream);
cudaError_t configure_colour_kernel();            // pic_colour.cuh (part of pic_render.cu)
cudaError_t launch_colour_kernel(const RenderParams& P, long long n_views, bool antialias, cudaStream_t stream);

size_t max_smem_bytes() { return render_smem_bytes() > sizeof(ExhaustiveSmem) ? render_smem_bytes() : sizeof(ExhaustiveSmem); }

cudaError_t configure_kernels() {
    cudaError_t err = configure_render_kernel();
    if (err != cudaSuccess) return err;
    err = configure_colour_kernel();
    if (err != cudaSuccess) return err;
    return cudaFuncSetAttribute(render_brute_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ExhaustiveSmem));
}

static RigParams rig_params(const RenderParams& P) {
    RigParams R;
    R.K = P.K; R.W = P.W; R.H = P.H; R.far_z = P.far_z; R.cls_sky = P.cls_sky; R.cls_ground = P.cls_ground;
    for (int k = 0; k < MAX_CAMS; ++k) R.cam[k] = P.cam[k];
    return R;
}

// Per call: rig tables, then agents (+ optional bicycle step) and their cameras.
cudaError_t launch_setup(const RenderParams& P, int n_agents, const float* poses, float* state, const float* actions,
                         const float* dims, const uint8_t* active, const uint8_t* agent_cls, AgentGeom* agents_out, ViewCam* cams_out,
                         float* tables, uint32_t* status, float dt, float wheelbase, float v_max, cudaStream_t stream) {
    const RigParams R = rig_params(P);
    float* ray_x = tables;
    float* ray_y = ray_x + (size_t)P.K * P.W;
    float* bg_z = ray_y + (size_t)P.K * P.H;
    uint32_t* bg_cls = reinterpret_cast<uint32_t*>(bg_z + (size_t)P.K * P.H);
    rig_kernel<<<P.K, 256, 0, stream>>>(R, ray_x, ray_y, bg_z, bg_cls, P.overflow);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess || n_agents <= 0) return err;
    agent_kernel<<<(n_agents + 127) / 128, 128, 0, stream>>>(n_agents, poses, state, actions, dims, active, agent_cls, P.cls_agent, agents_out,
                                                              cams_out, status, R, dt, wheelbase, v_max);
    return cudaGetLastError();
}

cudaError_t launch_colour(const RenderParams& P, long long n_views, bool antialias, cudaStream_t stream) {
    return n_views <= 0 ? cudaSuccess : launch_colour_kernel(P, n_views, antialias, stream);
}

cudaError_t launch_render(const RenderParams& P, long long n_views, bool brute, int sm_count, cudaStream_t stream) {
    if (n_views <= 0) return cudaSuccess;
    if (!brute) return launch_render_kernel(P, n_views, sm_count, stream);
    const long long blocks = n_views * P.tiles_x * P.tiles_y;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    render_brute_kernel<<<(unsigned)blocks, EXH_THREADS, sizeof(ExhaustiveSmem), stream>>>(P);
    const cudaError_t err = cudaGetLastError();
    return err != cudaSuccess ? err : launch_coverage_kernel(P, n_views, stream);
}

}  // namespace pic
