// Exhaustive tile renderer shared by the cross-check kernel (PIC_OPT_BRUTE_FORCE) and by
// pic_render_static (internal).
//
// One CTA renders one 64 x 64 tile of one view: every map item and every face of every other
// agent's box against every pixel (a thread per primitive, a shared-memory atomic max per
// fragment) -- no hierarchy, no frustum or pixel-box culling, no size classes.  It shares only the
// per-primitive arithmetic of pic_device.cuh (and the per-call camera and ray tables) with the
// production kernels, so comparing the images checks everything the production kernels add.
// The two users differ in where a map item comes from, which `fetch` hides: the scene's
// preprocessed primitives, or the caller's raw triangles.
#pragma once
#include "pic_device.cuh"

namespace pic {

constexpr int EXH_THREADS = 128;

struct __align__(16) ExhaustiveSmem {
    unsigned long long key[TILE * TILE];      // key = bits(1/z) << 32 | (0xFFFFFF - index) << 8 | class; 0 = background
    float ray_x[TILE], ray_y[TILE];
    Cam cam;
};

// fetch(i, cam, V, Pn, quad, flags, key_lo): map item i in camera space with its plane normal.
// n_map_tris: triangles of the map as given (box primitive indices start there).
template <class Fetch>
__device__ __forceinline__ void exhaustive_tile(ExhaustiveSmem& s, const RenderParams& P, unsigned job, uint32_t n_map_items,
                                                uint32_t n_map_tris, Fetch fetch) {
    const unsigned tiles = (unsigned)(P.tiles_x * P.tiles_y);
    const size_t view = (size_t)P.view_first + job / tiles;
    const int tile = (int)(job % tiles);
    const int k = (int)(view % (unsigned)P.K);
    const int a = (int)((view / (unsigned)P.K) % (unsigned)P.A);
    const int e = (int)(view / ((size_t)P.K * P.A));
    TileCtx t;
    t.x0 = (tile % P.tiles_x) * TILE; t.y0 = (tile / P.tiles_x) * TILE;
    t.tw = min(TILE, P.W - t.x0); t.th = min(TILE, P.H - t.y0);
    t.w_near = P.w_near; t.w_far = P.w_far; t.near_z = P.near_z; t.far_z = P.far_z;
    const AgentGeom ego = P.agents[(size_t)e * P.A + a];
    if (threadIdx.x == 0) load_camera(s.cam, P.cams[view], P.cam[k], P.W, P.H);
    for (int i = threadIdx.x; i < TILE * TILE; i += EXH_THREADS) s.key[i] = 0ull;
    if (threadIdx.x < TILE) {
        const int i = threadIdx.x;
        s.ray_x[i] = (t.x0 + i < P.W) ? P.rig.ray_x[(size_t)k * P.W + t.x0 + i] : 0.f;
        s.ray_y[i] = (t.y0 + i < P.H) ? P.rig.ray_y[(size_t)k * P.H + t.y0 + i] : 0.f;
    }
    __syncthreads();
    const Cam& c = s.cam;
    if (ego.active) {
        const uint32_t n_items = n_map_items + 6u * (uint32_t)P.A;
        for (uint32_t i = threadIdx.x; i < n_items; i += EXH_THREADS) {
            V3 V[4], Pn; bool quad; uint32_t flags, key_lo;
            if (i < n_map_items) {
                fetch(i, c, V, Pn, quad, flags, key_lo);
            } else {
                const uint32_t j = i - n_map_items;
                const int b = (int)(j / 6u), f = (int)(j % 6u);
                if (b == a) continue;
                const AgentGeom g = P.agents[(size_t)e * P.A + b];
                if (!g.active) continue;
                const uint32_t corners = face_corners(f);
#pragma unroll
                for (int q = 0; q < 4; ++q) V[q] = box_corner(c, g, (corners >> (4 * q)) & 7u);
                quad = true; flags = face_flags(corners);
                key_lo = ((0xFFFFFFu - (n_map_tris + 12u * (uint32_t)b + 2u * (uint32_t)f)) << 8) | agent_box_class(g);
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
    // keys -> images (scalar stores; this is a cross-check / small-batch path, not the fast one)
    const size_t img = (size_t)P.H * P.W;
    uint8_t* oc = P.out_class + view * img;
    uint16_t* od = P.out_depth + view * img;
    float* o32 = P.out_depth32 ? P.out_depth32 + view * img : nullptr;
    for (int i = threadIdx.x; i < t.th * t.tw; i += EXH_THREADS) {
        const int y = i / t.tw, x = i % t.tw;
        uint32_t cls = P.cls_sky; float z = P.far_z;
        if (ego.active) { cls = P.rig.bg_cls[(size_t)k * P.H + t.y0 + y]; z = P.rig.bg_z[(size_t)k * P.H + t.y0 + y]; }
        const unsigned long long key = s.key[y * TILE + x];
        if (P.occlusion) count_visible(P.occlusion + view * (size_t)P.A * 2u, key, n_map_tris);
        if (key) { cls = (uint32_t)(key & 0xff); z = fast_rcp(__uint_as_float((uint32_t)(key >> 32))); }
        const size_t o = (size_t)(t.y0 + y) * P.W + t.x0 + x;
        oc[o] = (uint8_t)cls;
        od[o] = __half_as_ushort(__float2half_rn(z));
        if (o32) o32[o] = z;
    }
}

}  // namespace pic
