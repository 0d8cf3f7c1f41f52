// Device-side arithmetic shared by every kernel of the rasterizer (internal).
//
// Everything that decides a pixel -- camera transform, edge functions, reciprocal-depth plane,
// coverage and depth test -- lives here and is written with explicit round-to-nearest intrinsics,
// so the production kernel and the exhaustive cross-check kernel evaluate bit-identical
// expressions for a given (primitive, pixel).
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "pic_types.h"

namespace pic {

constexpr float ZPROJ_FRAC = 0.5f;     // vertices nearer than this * near are not projected

// Geometry of the tile being rendered.
struct TileCtx {
    int x0, y0, tw, th;          // tile origin and size in pixels
    float w_near, w_far, near_z, far_z;
};

// Camera of one view: world -> camera rotation, origin and intrinsics.
struct __align__(16) Cam {
    float px, py;              // ego position
    float mwx, mwy, mwz;       // mount in world axes
    float rx, ry;              // right   (rz = 0)
    float dx, dy, dz;          // down
    float fx_, fy_, fz_;       // forward
    float focx, focy;          // focal lengths
    float cx, cy;              // principal point
};

struct PrimEq {
    float nx[4], ny[4], nz[4];   // E_i = nx*rx + ny*ry + nz, sign-normalised (inside: E_i > 0)
    float wx, wy, wz;            // 1/z = wx*rx + wy*ry + wz
    uint32_t tl;                 // bit i: exact zeros of edge i belong to the primitive
};

struct V3 { float x, y, z; };

__device__ __forceinline__ float fm(float a, float b, float c) { return __fmaf_rn(a, b, c); }
__device__ __forceinline__ float mul(float a, float b) { return __fmul_rn(a, b); }
__device__ __forceinline__ float sub(float a, float b) { return __fsub_rn(a, b); }
__device__ __forceinline__ float add(float a, float b) { return __fadd_rn(a, b); }

__device__ __forceinline__ V3 vsub(V3 a, V3 b) { return {sub(a.x, b.x), sub(a.y, b.y), sub(a.z, b.z)}; }
__device__ __forceinline__ V3 vcross(V3 a, V3 b) {
    return {fm(a.y, b.z, -mul(a.z, b.y)), fm(a.z, b.x, -mul(a.x, b.z)), fm(a.x, b.y, -mul(a.y, b.x))};
}
__device__ __forceinline__ float vdot(V3 a, V3 b) { return fm(a.x, b.x, fm(a.y, b.y, mul(a.z, b.z))); }

// World point -> camera space: subtract the ego position first (keeps float32 accurate far from
// the origin), then the mount, then rotate.
__device__ __forceinline__ V3 to_camera(const Cam& c, float X, float Y, float Z) {
    float qx = sub(sub(X, c.px), c.mwx);
    float qy = sub(sub(Y, c.py), c.mwy);
    float qz = sub(Z, c.mwz);
    V3 r;
    r.x = fm(c.rx, qx, mul(c.ry, qy));
    r.y = fm(c.dx, qx, fm(c.dy, qy, mul(c.dz, qz)));
    r.z = fm(c.fx_, qx, fm(c.fy_, qy, mul(c.fz_, qz)));
    return r;
}

// Ego-relative vector (already minus ego position) -> camera space, without the mount offset.
__device__ __forceinline__ V3 rotate_to_camera(const Cam& c, float qx, float qy, float qz) {
    V3 r;
    r.x = fm(c.rx, qx, mul(c.ry, qy));
    r.y = fm(c.dx, qx, fm(c.dy, qy, mul(c.dz, qz)));
    r.z = fm(c.fx_, qx, fm(c.fy_, qy, mul(c.fz_, qz)));
    return r;
}

// Camera of agent `ego` and rig camera `k`: heading + camera yaw by angle addition, mount turned
// into world axes, rotation rows (right, down, forward).
__device__ __forceinline__ void make_view_cam(ViewCam& c, const AgentGeom& ego, const CamConst& k) {
    const float ca = fm(ego.c, k.cpsi, -mul(ego.s, k.spsi));
    const float sa = fm(ego.s, k.cpsi, mul(ego.c, k.spsi));
    c.px = ego.x; c.py = ego.y;
    c.mwx = fm(ego.c, k.mx, -mul(ego.s, k.my));
    c.mwy = fm(ego.s, k.mx, mul(ego.c, k.my));
    c.mwz = k.mz;
    c.rx = sa; c.ry = -ca;
    c.fx = mul(k.cphi, ca); c.fy = mul(k.cphi, sa); c.fz = k.sphi;
    c.dx = mul(k.sphi, ca); c.dy = mul(k.sphi, sa); c.dz = -k.cphi;
    c.pad[0] = c.pad[1] = c.pad[2] = 0.f;
}

__device__ __forceinline__ void load_camera(Cam& c, const ViewCam& v, const CamConst& k, int W, int H) {
    c.px = v.px; c.py = v.py; c.mwx = v.mwx; c.mwy = v.mwy; c.mwz = v.mwz;
    c.rx = v.rx; c.ry = v.ry; c.dx = v.dx; c.dy = v.dy; c.dz = v.dz;
    c.fx_ = v.fx; c.fy_ = v.fy; c.fz_ = v.fz;
    c.focx = k.fx; c.focy = k.fy;
    c.cx = 0.5f * (float)W; c.cy = 0.5f * (float)H;
}

// Plane normal of a primitive from its camera-space vertices (used for box faces, whose corners are
// a few metres apart).
__device__ __forceinline__ V3 plane_normal(const V3 (&V)[4], bool quad) {
    return quad ? vcross(vsub(V[2], V[0]), vsub(V[3], V[1])) : vcross(vsub(V[1], V[0]), vsub(V[2], V[0]));
}

// Plane normal of a map primitive: the cross product is taken between WORLD-space edge vectors
// (differences of nearby coordinates, exact to a float32 ulp of the edge) and then rotated into
// camera space.  Differencing camera-space vertices instead would carry the rounding of the
// vertex distance into the edge and tilt the plane of a small, distant primitive.
__device__ __forceinline__ V3 plane_normal_world(const Cam& c, const float (&v)[12], bool quad) {
    V3 d1, d2;
    if (quad) { d1 = {sub(v[6], v[0]), sub(v[7], v[1]), sub(v[8], v[2])}; d2 = {sub(v[9], v[3]), sub(v[10], v[4]), sub(v[11], v[5])}; }
    else      { d1 = {sub(v[3], v[0]), sub(v[4], v[1]), sub(v[5], v[2])}; d2 = {sub(v[6], v[0]), sub(v[7], v[1]), sub(v[8], v[2])}; }
    const V3 nw = vcross(d1, d2);
    return rotate_to_camera(c, nw.x, nw.y, nw.z);
}

// Edge functions and reciprocal-depth plane of a primitive given in camera space, with its plane
// normal P (same orientation as the vertex order).
// Returns false for degenerate / edge-on primitives (D == 0), which cover nothing.
__device__ __forceinline__ bool prim_equations(const V3 (&V)[4], bool quad, uint32_t flags, const V3 P, PrimEq& q) {
    const int n = quad ? 4 : 3;
    V3 N[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (i < n) {
            const V3 a = V[i];
            const V3 b = (i == 3 || (i == 2 && !quad)) ? V[0] : V[(i + 1) & 3];
            if ((flags >> (4 + i)) & 1u) {       // evaluate in the canonical direction b -> a, then negate
                V3 t = vcross(b, vsub(a, b));
                N[i] = {-t.x, -t.y, -t.z};
            } else {
                N[i] = vcross(a, vsub(b, a));
            }
        } else {
            N[i] = {0.f, 0.f, 1.f};              // triangles: a fourth edge that is always inside
        }
    }
    float D = vdot(P, V[0]);
    if (!(D != 0.f)) return false;               // also drops NaN
    const float s = D < 0.f ? -1.f : 1.f;
    uint32_t tl = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float sx = (i < n) ? mul(s, N[i].x) : 0.f, sy = (i < n) ? mul(s, N[i].y) : 0.f, sz = (i < n) ? mul(s, N[i].z) : 1.f;
        q.nx[i] = sx; q.ny[i] = sy; q.nz[i] = sz;
        if (sx > 0.f || (sx == 0.f && sy > 0.f)) tl |= 1u << i;
    }
    q.tl = tl;
    q.wx = __fdiv_rn(P.x, D); q.wy = __fdiv_rn(P.y, D); q.wz = __fdiv_rn(P.z, D);
    return true;
}

// Fragment of a primitive at the ray (rx, ry, 1): the high key word (bits of 1/z), or 0 if the
// pixel is not covered or the depth is outside [near, far].
__device__ __forceinline__ uint32_t fragment(const PrimEq& q, float rx, float ry, float w_near, float w_far) {
    bool in = true;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float e = fm(q.nx[i], rx, fm(q.ny[i], ry, q.nz[i]));
        // e > 0 || (e == 0 && the edge owns its zeros) as one comparison: nothing lies between the
        // smallest negative subnormal and zero, and neither fma nor the comparison flushes subnormals
        in = in && (e > __int_as_float(((q.tl >> i) & 1u) ? (int)0x80000001u : 0));
    }
    float w = fm(q.wx, rx, fm(q.wy, ry, q.wz));
    in = in && (w >= w_far) && (w <= w_near);
    return in ? __float_as_uint(w) : 0u;
}

// Counts a pixel won by a box face for its agent: the low key word holds 0xFFFFFF - primitive index,
// box primitives start at n_map_tris, 12 per agent.
__device__ __forceinline__ void count_visible(uint32_t* occ_view, unsigned long long key, uint32_t n_map_tris) {
    const uint32_t index = 0xFFFFFFu - ((uint32_t)key >> 8);
    if (key != 0ull && index >= n_map_tris) atomicAdd(occ_view + 2u * ((index - n_map_tris) / 12u), 1u);
}

__device__ __forceinline__ unsigned long long make_key(uint32_t wbits, uint32_t key_lo) {
    return ((unsigned long long)wbits << 32) | key_lo;
}


// Pixel box (inclusive, tile coordinates) of camera-space vertices, or the whole tile when a
// vertex is too close to the camera plane to project.  Returns false if the primitive cannot
// touch any pixel centre of the tile (with the default margin m) or lies entirely before near / beyond far.
// (Triangles pass their third vertex twice.)
__device__ __forceinline__ bool pixel_box(const Cam& c, const TileCtx& t, const V3 (&V)[4], uint32_t& packed, const float m = 0.00390625f) {
    constexpr int n = 4;
    float zmin = V[0].z, zmax = V[0].z;
#pragma unroll
    for (int i = 1; i < n; ++i) { zmin = fminf(zmin, V[i].z); zmax = fmaxf(zmax, V[i].z); }
    // (written without early exits: the lanes of a warp rarely agree, so exits save nothing)
    bool ok = (zmax >= t.near_z * 0.9999f) && (zmin <= t.far_z * 1.0001f);
    int bx0 = 0, by0 = 0, bx1 = t.tw - 1, by1 = t.th - 1;
    if (zmin >= t.near_z * ZPROJ_FRAC) {
        float sx0 = 3e38f, sx1 = -3e38f, sy0 = 3e38f, sy1 = -3e38f;
#pragma unroll
        for (int i = 0; i < n; ++i) {
            float iz = __fdividef(1.0f, V[i].z);
            float sx = fm(c.focx, mul(V[i].x, iz), c.cx), sy = fm(c.focy, mul(V[i].y, iz), c.cy);
            sx0 = fminf(sx0, sx); sx1 = fmaxf(sx1, sx); sy0 = fminf(sy0, sy); sy1 = fmaxf(sy1, sy);
        }
        // pixel centres u + 0.5 in [sx0, sx1], widened by m = 1/256 pixel against rounding (m = 1/2 + 1/256: every pixel
        // whose unit square the primitive touches)
        float fx0 = ceilf(sx0 - 0.5f - m) - (float)t.x0, fx1 = floorf(sx1 - 0.5f + m) - (float)t.x0;
        float fy0 = ceilf(sy0 - 0.5f - m) - (float)t.y0, fy1 = floorf(sy1 - 0.5f + m) - (float)t.y0;
        ok = ok && (fx0 <= fx1) && (fy0 <= fy1) && (fx1 >= 0.f) && (fy1 >= 0.f) && (fx0 <= (float)(t.tw - 1)) && (fy0 <= (float)(t.th - 1));
        bx0 = (int)fmaxf(fx0, 0.f); by0 = (int)fmaxf(fy0, 0.f);
        bx1 = (int)fminf(fx1, (float)(t.tw - 1)); by1 = (int)fminf(fy1, (float)(t.th - 1));
    } else if (ok) {
        // frustum side planes through the camera centre, valid for any sign of z
        float l = (float)t.x0 - c.cx, r = (float)(t.x0 + t.tw) - c.cx, u = (float)t.y0 - c.cy, d = (float)(t.y0 + t.th) - c.cy;
        bool ol = true, orr = true, ou = true, od = true;
#pragma unroll
        for (int i = 0; i < n; ++i) {
            float X = mul(V[i].x, c.focx), Y = mul(V[i].y, c.focy), Z = V[i].z;
            ol = ol && (X < mul(Z, l) - 1e-4f * (fabsf(X) + fabsf(mul(Z, l))));
            orr = orr && (X > mul(Z, r) + 1e-4f * (fabsf(X) + fabsf(mul(Z, r))));
            ou = ou && (Y < mul(Z, u) - 1e-4f * (fabsf(Y) + fabsf(mul(Z, u))));
            od = od && (Y > mul(Z, d) + 1e-4f * (fabsf(Y) + fabsf(mul(Z, d))));
        }
        ok = !(ol || orr || ou || od);
    }
    packed = (uint32_t)bx0 | ((uint32_t)by0 << 8) | ((uint32_t)bx1 << 16) | ((uint32_t)by1 << 24);
    return ok;
}


__device__ __forceinline__ void load_prim(const Prim* __restrict__ p, float (&v)[12], uint32_t& key_lo, uint32_t& flags, float& vis_cos) {
    const float4* q = reinterpret_cast<const float4*>(p);
    float4 a = __ldg(q), b = __ldg(q + 1), c = __ldg(q + 2);
    uint4 d = __ldg(reinterpret_cast<const uint4*>(q + 3));
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    v[8] = c.x; v[9] = c.y; v[10] = c.z; v[11] = c.w;
    key_lo = d.x; flags = d.y; vis_cos = __uint_as_float(d.z);
}
__device__ __forceinline__ void load_prim(const Prim* __restrict__ p, float (&v)[12], uint32_t& key_lo, uint32_t& flags) {
    float vis_cos;
    load_prim(p, v, key_lo, flags, vis_cos);
}

// A triangle with vis_cos > 0 is drawn only from its front side and only if the direction from its
// centroid to the camera (the origin of camera space) is within acos(vis_cos) of its normal P (by
// vertex order).  Outside that range its plane normal is replaced by zero, which makes
// prim_equations reject it as degenerate -- so every kernel that sets a primitive up drops it alike.
__device__ __forceinline__ V3 limit_angular_range(const V3 (&V)[4], V3 P, float vis_cos) {
    if (vis_cos > 0.f) {
        const V3 g = {add(add(V[0].x, V[1].x), V[2].x), add(add(V[0].y, V[1].y), V[2].y), add(add(V[0].z, V[1].z), V[2].z)};   // 3 x centroid
        const float s = -vdot(P, g);
        const float pp = vdot(P, P), gg = vdot(g, g);
        const bool in = s >= 0.f && mul(s, s) >= mul(mul(vis_cos, vis_cos), mul(pp, gg));
        if (!in) P = {0.f, 0.f, 0.f};
    }
    return P;
}

// Class of an agent's box (AgentGeom::active = 1 | class << 8).
__device__ __forceinline__ uint32_t agent_box_class(const AgentGeom& g) { return (g.active >> 8) & 0xffu; }

// Box corner i (bit0 +x, bit1 +y, bit2 top) of agent g in camera space.
__device__ __forceinline__ V3 box_corner(const Cam& c, const AgentGeom& g, int i) {
    float sx = (i & 1) ? g.hl : -g.hl, sy = (i & 2) ? g.hw : -g.hw;
    float qx = add(sub(g.x, c.px), fm(g.c, sx, -mul(g.s, sy)));
    float qy = add(sub(g.y, c.py), fm(g.s, sx, mul(g.c, sy)));
    float qz = (i & 4) ? g.h : 0.f;
    return rotate_to_camera(c, sub(qx, c.mwx), sub(qy, c.mwy), sub(qz, c.mwz));
}

// Faces of a box as corner quadruples in perimeter order, one nibble per corner:
// rear (-x), front (+x), right (-y), left (+y), bottom, top.
__device__ __forceinline__ uint32_t face_corners(int f) {
    const uint32_t tab[6] = {0x4620u, 0x3751u, 0x1540u, 0x6732u, 0x2310u, 0x5764u};
    uint32_t r = tab[0];
#pragma unroll
    for (int i = 1; i < 6; ++i) r = (f == i) ? tab[i] : r;
    return r;
}

__device__ __forceinline__ uint32_t face_flags(uint32_t corners) {
    uint32_t fl = 1u;   // quad
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t a = (corners >> (4 * k)) & 7u, b = (corners >> (4 * ((k + 1) & 3))) & 7u;
        if (!(a < b)) fl |= 1u << (4 + k);     // canonical direction: lower corner index first
    }
    return fl;
}

// Background of an image row with ray coordinate ry for a camera with pitch (cphi, sphi) mounted
// mz above the ground: the analytic ground plane z = 0 below the horizon (depth clamped to far),
// sky above.
__device__ __forceinline__ void background(float cphi, float sphi, float mz, float ry, float far_z, uint32_t cls_sky,
                                           uint32_t cls_ground, uint32_t& cls, float& z) {
    const float wr = fm(-ry, cphi, sphi);          // world-z component of the ray
    cls = cls_sky; z = far_z;
    if (wr < 0.f && mz > 0.f) { cls = cls_ground; z = fminf(far_z, __fdiv_rn(mz, -wr)); }
}

__device__ __forceinline__ float fast_rcp(float x) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

}  // namespace pic
