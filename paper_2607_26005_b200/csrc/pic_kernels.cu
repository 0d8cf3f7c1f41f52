// CUDA kernels of the batched egocentric rasterizer (sm_100a).
//
// One CTA renders one tile (up to 64 x 64 pixels) of one view.  The z-buffer lives in shared
// memory as one 64-bit key per pixel:
//     key = float_bits(1/z) << 32 | (0xFFFFFF - primitive index) << 8 | class
// so "nearest fragment wins, ties to the lower index" is a plain unsigned max, independent of
// the order in which primitives are processed; 0 means "no fragment" (background).
//
// Steps per tile:
//   (a) cull      group boxes -> leaf boxes (compacted with warp ballots) -> primitives against the
//                 tile frustum and the pixel grid; other agents' boxes are culled as spheres and
//                 only their camera-facing faces are kept
//   (c) set-up    per survivor: camera-space vertices, 3-4 edge functions, 1/z plane
//       tiny      primitives whose pixel box holds <= 4 pixel centres are rasterized at once by
//                 their thread with a shared-memory atomic max
//       medium    pixel boxes up to 64 centres: one warp per primitive, a lane per pixel, atomic max
//   (b) binning   larger ones are tested against the 8 x 8 pixel blocks of the tile (trivial
//                 reject / trivial accept with the same float32 edge functions) into bit masks
//   (c) raster    each warp owns blocks; a lane owns two pixels, keeps their keys in registers
//                 and walks the block's mask
//   (d) store     keys -> class u8 + depth binary16, 16 pixels per thread, 128-bit stores
//
// All arithmetic that decides a pixel is written with explicit round-to-nearest intrinsics so that
// every kernel (production and exhaustive) evaluates bit-identical expressions.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "pic_types.h"

namespace pic {

constexpr int NW = NTHREADS / 32;
constexpr int LCAP = 64;          // binned (large) primitives per tile pass: one mask bit each
constexpr int MCAP = 64;          // medium primitives (warp-cooperative raster) per tile pass
constexpr int GROUP_BATCH = 16;   // groups examined per batch
constexpr int LEAFCAP = GROUP_BATCH * GROUP_LEAVES;   // visible leaves per batch
constexpr int FACECAP = 6 * NTHREADS;                 // box-face items per round of NTHREADS boxes
constexpr int REC = 17;           // words per set-up record (odd: conflict-free per-lane reads)
constexpr int TINY_MAX_PIXELS = 4;     // pixel centres in the box of a primitive rasterized by its own thread
constexpr int MEDIUM_MAX_PIXELS = 64;  // ... rasterized by one warp with atomics; larger ones are binned
constexpr float ZPROJ_FRAC = 0.5f;     // vertices nearer than this * near are not projected

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

__device__ __forceinline__ void make_camera(Cam& c, const AgentGeom& ego, const CamConst& k, int W, int H) {
    float ca = fm(ego.c, k.cpsi, -mul(ego.s, k.spsi));
    float sa = fm(ego.s, k.cpsi, mul(ego.c, k.spsi));
    c.px = ego.x; c.py = ego.y;
    c.mwx = fm(ego.c, k.mx, -mul(ego.s, k.my));
    c.mwy = fm(ego.s, k.mx, mul(ego.c, k.my));
    c.mwz = k.mz;
    c.rx = sa; c.ry = -ca;
    c.fx_ = mul(k.cphi, ca); c.fy_ = mul(k.cphi, sa); c.fz_ = k.sphi;
    c.dx = mul(k.sphi, ca); c.dy = mul(k.sphi, sa); c.dz = -k.cphi;
    c.focx = k.fx; c.focy = k.fy;
    c.cx = 0.5f * (float)W; c.cy = 0.5f * (float)H;
}

// Edge functions and reciprocal-depth plane of a primitive given in camera space.
// Returns false for degenerate / edge-on primitives (D == 0), which cover nothing.
__device__ __forceinline__ bool prim_equations(const V3 (&V)[4], bool quad, uint32_t flags, PrimEq& q) {
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
    V3 P = quad ? vcross(vsub(V[2], V[0]), vsub(V[3], V[1])) : vcross(vsub(V[1], V[0]), vsub(V[2], V[0]));
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
        in = in && (e > 0.f || (e == 0.f && ((q.tl >> i) & 1u)));
    }
    float w = fm(q.wx, rx, fm(q.wy, ry, q.wz));
    in = in && (w >= w_far) && (w <= w_near);
    return in ? __float_as_uint(w) : 0u;
}

__device__ __forceinline__ unsigned long long make_key(uint32_t wbits, uint32_t key_lo) {
    return ((unsigned long long)wbits << 32) | key_lo;
}

// ------------------------------------------------------------------------------------------------
// agent kernel: poses/dims/active -> AgentGeom (optionally after one kinematic-bicycle step)
// ------------------------------------------------------------------------------------------------
__global__ void agent_kernel(int n, const float* __restrict__ poses, int pose_stride, float* state,
                             const float* __restrict__ actions, const float* __restrict__ dims,
                             const uint8_t* __restrict__ active, AgentGeom* __restrict__ out, uint32_t* status,
                             float dt, float wheelbase, float v_max) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    bool act = active ? active[i] != 0 : true;
    float x, y, th;
    if (state) {                                   // pic_step: update the scene's own state in place
        float v;
        x = state[4 * i]; y = state[4 * i + 1]; th = state[4 * i + 2]; v = state[4 * i + 3];
        if (actions && act) {
            float acc = actions[2 * i], steer = actions[2 * i + 1];
            float s, c;
            sincosf(th, &s, &c);
            float nx = fm(mul(v, c), dt, x);
            float ny = fm(mul(v, s), dt, y);
            float nth = fm(mul(__fdiv_rn(v, wheelbase), tanf(steer)), dt, th);
            float nv = fminf(fmaxf(fm(acc, dt, v), 0.f), v_max);
            x = nx; y = ny; th = nth; v = nv;
            state[4 * i] = x; state[4 * i + 1] = y; state[4 * i + 2] = th; state[4 * i + 3] = v;
        }
    } else {
        x = poses[pose_stride * i]; y = poses[pose_stride * i + 1]; th = poses[pose_stride * i + 2];
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
    g.active = act ? 1u : 0u;
    out[i] = g;
}


// ------------------------------------------------------------------------------------------------
// shared-memory layout of a render CTA
// ------------------------------------------------------------------------------------------------
struct __align__(16) TileSmem {
    unsigned long long key[TILE * TILE];      // 32 KB, 16-byte chunks XOR-swizzled by row (key_index)
    float rec_l[LCAP * REC];                  // set-up records of binned primitives
    float rec_m[MCAP * REC];                  // set-up records of medium primitives
    unsigned long long bin_any[64];           // per 8x8 block: binned primitives to test
    unsigned long long bin_full[64];          // per 8x8 block: primitives covering the whole block, depth in range
    union {
        uint32_t leaf[LEAFCAP];               // visible leaves of the batch: first primitive << 4 | count
        uint32_t face[LEAFCAP];               // box-face items: agent << 3 | face
    };
    uint32_t grp[GROUP_BATCH];
    float ray_x[TILE], ray_y[TILE];           // ray coordinates of the tile's pixel columns / rows
    float plane[6][4];                        // tile frustum, ego-relative world space, unit normals: n, offset
    float side[4][4];                         // the four side planes in camera space, unit normals
    Cam cam;
    int n_large, n_med, n_leaf, n_grp, n_face;
    uint32_t touched[2];                      // 8x8 blocks that may hold a fragment (rows 0-3, rows 4-7)
    unsigned long long cnt[16];
};

struct TileCtx {
    int x0, y0, tw, th;          // tile origin and size in pixels
    float w_near, w_far, near_z, far_z;
    int med_cap, large_cap;
};

// Keys are stored so that both an 8x8 block (raster) and 16-pixel row segments (store) spread over
// all banks: the 16-byte chunk holding pixels (2c, 2c+1) of row y sits at chunk c ^ (y & 7).
__device__ __forceinline__ int key_index(int x, int y) {
    return (y << 6) | ((((x >> 1) ^ (y & 7)) << 1) | (x & 1));
}

// Bit mask of the 8x8 blocks touched by a pixel box (inclusive).
__device__ __forceinline__ unsigned long long block_mask(int bx0, int by0, int bx1, int by1) {
    const int c0 = bx0 >> 3, c1 = bx1 >> 3, r0 = by0 >> 3, r1 = by1 >> 3;
    const unsigned long long row = (unsigned long long)(((2u << c1) - (1u << c0)) & 0xffu);
    const unsigned long long rows = (0x0101010101010101ull >> (8 * (7 - (r1 - r0)))) << (8 * r0);
    return row * rows;
}

__device__ __forceinline__ void mark_touched(TileSmem& s, unsigned long long m) {
    const uint32_t lo = (uint32_t)m, hi = (uint32_t)(m >> 32);
    if (lo & ~s.touched[0]) atomicOr(&s.touched[0], lo);
    if (hi & ~s.touched[1]) atomicOr(&s.touched[1], hi);
}

// Is the box [lo,hi] (world) possibly inside the tile frustum?  Conservative.
__device__ __forceinline__ bool box_visible(const TileSmem& s, const Node& b) {
    const float ax = sub(b.lo[0], s.cam.px), bx = sub(b.hi[0], s.cam.px);
    const float ay = sub(b.lo[1], s.cam.py), by = sub(b.hi[1], s.cam.py);
    const float cx = 0.5f * (ax + bx), cy = 0.5f * (ay + by), cz = 0.5f * (b.lo[2] + b.hi[2]);
    const float hx = 0.5f * (bx - ax), hy = 0.5f * (by - ay), hz = 0.5f * (b.hi[2] - b.lo[2]);
    // rounding of the few float32 operations below, far under any real distance
    const float slack = 1e-3f + 4e-6f * (fabsf(cx) + fabsf(cy) + fabsf(cz) + hx + hy + hz);
    bool vis = true;
#pragma unroll
    for (int p = 0; p < 6; ++p) {
        const float nx = s.plane[p][0], ny = s.plane[p][1], nz = s.plane[p][2], d = s.plane[p][3];
        const float dist = nx * cx + ny * cy + nz * cz + d;
        const float reach = fabsf(nx) * hx + fabsf(ny) * hy + fabsf(nz) * hz;
        vis = vis && (dist + reach >= -slack);
    }
    return vis;
}

// Pixel box (inclusive, tile coordinates) of camera-space vertices, or the whole tile when a
// vertex is too close to the camera plane to project.  Returns false if the primitive cannot
// touch any pixel centre of the tile or lies entirely before near / beyond far.
// (Triangles pass their third vertex twice.)
__device__ __forceinline__ bool pixel_box(const Cam& c, const TileCtx& t, const V3 (&V)[4], uint32_t& packed) {
    constexpr int n = 4;
    float zmin = V[0].z, zmax = V[0].z;
#pragma unroll
    for (int i = 1; i < n; ++i) { zmin = fminf(zmin, V[i].z); zmax = fmaxf(zmax, V[i].z); }
    if (!(zmax >= t.near_z * 0.9999f) || !(zmin <= t.far_z * 1.0001f)) return false;
    int bx0 = 0, by0 = 0, bx1 = t.tw - 1, by1 = t.th - 1;
    if (zmin >= t.near_z * ZPROJ_FRAC) {
        float sx0 = 3e38f, sx1 = -3e38f, sy0 = 3e38f, sy1 = -3e38f;
#pragma unroll
        for (int i = 0; i < n; ++i) {
            float iz = __fdividef(1.0f, V[i].z);
            float sx = fm(c.focx, mul(V[i].x, iz), c.cx), sy = fm(c.focy, mul(V[i].y, iz), c.cy);
            sx0 = fminf(sx0, sx); sx1 = fmaxf(sx1, sx); sy0 = fminf(sy0, sy); sy1 = fmaxf(sy1, sy);
        }
        // pixel centres u + 0.5 in [sx0, sx1], widened by 1/256 pixel against rounding
        const float m = 0.00390625f;
        float fx0 = ceilf(sx0 - 0.5f - m) - (float)t.x0, fx1 = floorf(sx1 - 0.5f + m) - (float)t.x0;
        float fy0 = ceilf(sy0 - 0.5f - m) - (float)t.y0, fy1 = floorf(sy1 - 0.5f + m) - (float)t.y0;
        if (!(fx0 <= fx1) || !(fy0 <= fy1)) return false;
        if (fx1 < 0.f || fy1 < 0.f || fx0 > (float)(t.tw - 1) || fy0 > (float)(t.th - 1)) return false;
        bx0 = (int)fmaxf(fx0, 0.f); by0 = (int)fmaxf(fy0, 0.f);
        bx1 = (int)fminf(fx1, (float)(t.tw - 1)); by1 = (int)fminf(fy1, (float)(t.th - 1));
    } else {
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
        if (ol || orr || ou || od) return false;
    }
    packed = (uint32_t)bx0 | ((uint32_t)by0 << 8) | ((uint32_t)bx1 << 16) | ((uint32_t)by1 << 24);
    return true;
}

__device__ __forceinline__ void load_prim(const Prim* __restrict__ p, float (&v)[12], uint32_t& key_lo, uint32_t& flags) {
    const float4* q = reinterpret_cast<const float4*>(p);
    float4 a = __ldg(q), b = __ldg(q + 1), c = __ldg(q + 2);
    uint4 d = __ldg(reinterpret_cast<const uint4*>(q + 3));
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    v[8] = c.x; v[9] = c.y; v[10] = c.z; v[11] = c.w;
    key_lo = d.x; flags = d.y;
}

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

// Rasterize a primitive from one thread: loop over its pixel box, atomic max per fragment.
__device__ __forceinline__ int raster_in_thread(TileSmem& s, const TileCtx& t, const PrimEq& q, uint32_t key_lo, uint32_t box) {
    const int bx0 = box & 0xff, by0 = (box >> 8) & 0xff, bx1 = (box >> 16) & 0xff, by1 = box >> 24;
    int frags = 0;
    for (int y = by0; y <= by1; ++y) {
        const float ry = s.ray_y[y];
        for (int x = bx0; x <= bx1; ++x) {
            const uint32_t wb = fragment(q, s.ray_x[x], ry, t.w_near, t.w_far);
            if (wb) {
                const unsigned long long k = make_key(wb, key_lo);
                unsigned long long* addr = &s.key[key_index(x, y)];
                if (k > *reinterpret_cast<volatile unsigned long long*>(addr)) atomicMax(addr, k);
                ++frags;
            }
        }
    }
    if (frags) mark_touched(s, block_mask(bx0, by0, bx1, by1));
    return frags;
}

__device__ __forceinline__ void store_record(float* r, const PrimEq& q, uint32_t key_lo, uint32_t box) {
#pragma unroll
    for (int i = 0; i < 4; ++i) { r[i] = q.nx[i]; r[4 + i] = q.ny[i]; r[8 + i] = q.nz[i]; }
    r[12] = q.wx; r[13] = q.wy; r[14] = q.wz;
    r[15] = __uint_as_float(key_lo);
    // the pixel box needs 6 bits per coordinate; the top-left bits ride along
    const uint32_t bx0 = box & 0xff, by0 = (box >> 8) & 0xff, bx1 = (box >> 16) & 0xff, by1 = box >> 24;
    r[16] = __uint_as_float(bx0 | (by0 << 6) | (bx1 << 12) | (by1 << 18) | (q.tl << 24));
}

struct Tally { int tested, setup, tiny, medium, large, fallback, frags; };

// Cull one primitive against the tile, set it up, and route it by the size of its pixel box.
__device__ __forceinline__ void process_prim(TileSmem& s, const TileCtx& t, const V3 (&V)[4], bool quad, uint32_t flags,
                                             uint32_t key_lo, Tally& n) {
    ++n.tested;
    uint32_t box;
    if (!pixel_box(s.cam, t, V, box)) return;
    PrimEq q;
    if (!prim_equations(V, quad, flags, q)) return;
    ++n.setup;
    const int bx0 = box & 0xff, by0 = (box >> 8) & 0xff, bx1 = (box >> 16) & 0xff, by1 = box >> 24;
    const int area = (bx1 - bx0 + 1) * (by1 - by0 + 1);
    if (area <= TINY_MAX_PIXELS) {
        n.frags += raster_in_thread(s, t, q, key_lo, box);
        ++n.tiny;
        return;
    }
    if (area <= MEDIUM_MAX_PIXELS) {
        const int slot = atomicAdd(&s.n_med, 1);
        if (slot < t.med_cap) { store_record(&s.rec_m[slot * REC], q, key_lo, box); ++n.medium; return; }
    } else {
        const int slot = atomicAdd(&s.n_large, 1);
        if (slot < t.large_cap) { store_record(&s.rec_l[slot * REC], q, key_lo, box); ++n.large; return; }
    }
    // list full: correct but slow
    n.frags += raster_in_thread(s, t, q, key_lo, box);
    ++n.fallback;
}

// Medium primitives: one warp per primitive, lanes tile its pixel box 8 x 4 at a time.
__device__ int raster_medium(TileSmem& s, const TileCtx& t) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = min(s.n_med, t.med_cap);
    int frags = 0;
    for (int p = warp; p < n; p += NW) {
        const float* r = &s.rec_m[p * REC];
        PrimEq q;
#pragma unroll
        for (int i = 0; i < 4; ++i) { q.nx[i] = r[i]; q.ny[i] = r[4 + i]; q.nz[i] = r[8 + i]; }
        q.wx = r[12]; q.wy = r[13]; q.wz = r[14];
        const uint32_t key_lo = __float_as_uint(r[15]);
        const uint32_t bw = __float_as_uint(r[16]);
        q.tl = bw >> 24;
        const int bx0 = bw & 63, by0 = (bw >> 6) & 63, bx1 = (bw >> 12) & 63, by1 = (bw >> 18) & 63;
        bool any = false;
        for (int yy = by0; yy <= by1; yy += 4) {
            const int y = yy + (lane >> 3);
            for (int xx = bx0; xx <= bx1; xx += 8) {
                const int x = xx + (lane & 7);
                if (x <= bx1 && y <= by1) {
                    const uint32_t wb = fragment(q, s.ray_x[x], s.ray_y[y], t.w_near, t.w_far);
                    if (wb) {
                        const unsigned long long k = make_key(wb, key_lo);
                        unsigned long long* addr = &s.key[key_index(x, y)];
                        if (k > *reinterpret_cast<volatile unsigned long long*>(addr)) atomicMax(addr, k);
                        any = true;
                        ++frags;
                    }
                }
            }
        }
        if (__any_sync(0xffffffffu, any) && lane == 0) mark_touched(s, block_mask(bx0, by0, bx1, by1));
    }
    return frags;
}

// (b) binning: test every large primitive against the 8x8 blocks its pixel box touches.
// Work item = (primitive, block row).  The caller synchronises before and after.
__device__ void bin_large(TileSmem& s, const TileCtx& t) {
    const int n = min(s.n_large, t.large_cap);
    for (int item = threadIdx.x; item < n * 8; item += NTHREADS) {
        const int p = item >> 3, brow = item & 7;
        const float* r = &s.rec_l[p * REC];
        const uint32_t bw = __float_as_uint(r[16]);
        const int bx0 = bw & 63, by0 = (bw >> 6) & 63, bx1 = (bw >> 12) & 63, by1 = (bw >> 18) & 63;
        if (brow < (by0 >> 3) || brow > (by1 >> 3)) continue;
        // rows of this block row that exist in the tile
        const int ya = brow * 8, yb = min(brow * 8 + 7, t.th - 1);
        const float rya = s.ray_y[ya], ryb = s.ray_y[yb];
        float tmin[4], tmax[4], nx[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float ny = r[4 + e], nz = r[8 + e];
            const float ta = fm(ny, rya, nz), tb = fm(ny, ryb, nz);
            tmin[e] = fminf(ta, tb); tmax[e] = fmaxf(ta, tb);
            nx[e] = r[e];
        }
        const float wx = r[12], wy = r[13], wz = r[14];
        const float wa = fm(wy, rya, wz), wb = fm(wy, ryb, wz);
        const float wtmin = fminf(wa, wb), wtmax = fmaxf(wa, wb);
        unsigned long long any = 0ull, full = 0ull;
        for (int bcol = bx0 >> 3; bcol <= (bx1 >> 3); ++bcol) {
            const int xa = bcol * 8, xb = min(bcol * 8 + 7, t.tw - 1);
            const float rxa = s.ray_x[xa], rxb = s.ray_x[xb];    // rxa < rxb
            bool reject = false, inside = true;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                // fma is monotone in each argument, so the block's extreme values are at its corners
                const float emax = fm(nx[e], nx[e] >= 0.f ? rxb : rxa, tmax[e]);
                const float emin = fm(nx[e], nx[e] >= 0.f ? rxa : rxb, tmin[e]);
                reject = reject || (emax < 0.f);
                inside = inside && (emin > 0.f);
            }
            const float wmax = fm(wx, wx >= 0.f ? rxb : rxa, wtmax), wmin = fm(wx, wx >= 0.f ? rxa : rxb, wtmin);
            reject = reject || (wmax < t.w_far) || (wmin > t.w_near);
            inside = inside && (wmin >= t.w_far) && (wmax <= t.w_near);
            if (reject) continue;
            any |= 1ull << bcol;
            if (inside) full |= 1ull << bcol;
        }
        for (; any; any &= any - 1) {
            const int bcol = __ffsll((long long)any) - 1;
            atomicOr(&s.bin_any[brow * 8 + bcol], 1ull << p);
            if ((full >> bcol) & 1ull) atomicOr(&s.bin_full[brow * 8 + bcol], 1ull << p);
        }
    }
}

// (c) raster of the binned primitives: a warp owns an 8x8 block, a lane two horizontally adjacent
// pixels whose keys stay in registers while the block's primitives are walked.
__device__ int raster_large(TileSmem& s, const TileCtx& t) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int frags = 0;
    for (int blk = warp; blk < 64; blk += NW) {
        unsigned long long any = s.bin_any[blk];
        if (!any) continue;
        const unsigned long long fullm = s.bin_full[blk];
        const int x = (blk & 7) * 8 + (lane & 3) * 2, y = (blk >> 3) * 8 + (lane >> 2);
        const float rx0 = s.ray_x[x], rx1 = s.ray_x[x + 1], ry = s.ray_y[y];
        ulonglong2* kp = reinterpret_cast<ulonglong2*>(&s.key[key_index(x, y)]);
        ulonglong2 kk = *kp;
        while (any) {
            const int p = __ffsll((long long)any) - 1;
            any &= any - 1;
            const float* r = &s.rec_l[p * REC];
            const uint32_t key_lo = __float_as_uint(r[15]);
            const float wt = fm(r[13], ry, r[14]);
            const float w0 = fm(r[12], rx0, wt), w1 = fm(r[12], rx1, wt);
            bool in0 = true, in1 = true;
            if (!((fullm >> p) & 1ull)) {
                const uint32_t tl = __float_as_uint(r[16]) >> 24;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float te = fm(r[4 + e], ry, r[8 + e]);
                    const float e0 = fm(r[e], rx0, te), e1 = fm(r[e], rx1, te);
                    const bool own = (tl >> e) & 1u;
                    in0 = in0 && (e0 > 0.f || (e0 == 0.f && own));
                    in1 = in1 && (e1 > 0.f || (e1 == 0.f && own));
                }
                in0 = in0 && (w0 >= t.w_far) && (w0 <= t.w_near);
                in1 = in1 && (w1 >= t.w_far) && (w1 <= t.w_near);
            }
            if (in0) { const unsigned long long k = make_key(__float_as_uint(w0), key_lo); if (k > kk.x) kk.x = k; ++frags; }
            if (in1) { const unsigned long long k = make_key(__float_as_uint(w1), key_lo); if (k > kk.y) kk.y = k; ++frags; }
        }
        *kp = kk;
    }
    return frags;
}

__device__ __forceinline__ float fast_rcp(float x) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// (d) keys -> class / depth images.
__device__ void store_tile(const TileSmem& s, const TileCtx& t, const RenderParams& P, size_t view, bool ego_active) {
    const Cam& c = s.cam;
    const size_t img = (size_t)P.H * P.W;
    uint8_t* oc = P.out_class + view * img;
    uint16_t* od = P.out_depth + view * img;
    float* o32 = P.out_depth32 ? P.out_depth32 + view * img : nullptr;
    const float cphi = -c.dz, sphi = c.fz_;
    const bool vec = (t.tw % 16 == 0) && (P.W % 16 == 0) && o32 == nullptr;
    const int segs_per_row = (t.tw + 15) / 16;
    const unsigned long long touched = ((unsigned long long)s.touched[1] << 32) | s.touched[0];
    for (int seg = threadIdx.x; seg < t.th * segs_per_row; seg += NTHREADS) {
        const int y = seg / segs_per_row, xs = (seg % segs_per_row) * 16;
        // background of this row: analytic ground plane below the horizon, sky above
        const float wr = fm(-s.ray_y[y], cphi, sphi);
        uint32_t bg_cls = P.cls_sky;
        float bg_z = P.far_z;
        if (wr < 0.f && c.mwz > 0.f) { bg_cls = P.cls_ground; bg_z = fminf(P.far_z, __fdiv_rn(c.mwz, -wr)); }
        if (!ego_active) { bg_cls = P.cls_sky; bg_z = P.far_z; }
        const size_t o = (size_t)(t.y0 + y) * P.W + t.x0 + xs;
        const bool empty = ((touched >> ((y >> 3) * 8 + (xs >> 3))) & 3ull) == 0ull;   // both blocks of the segment
        if (vec) {
            uint32_t cw[4];
            uint32_t dw[8];
            if (empty) {
                const uint32_t c4 = bg_cls * 0x01010101u;
                const __half2 h = __floats2half2_rn(bg_z, bg_z);
                const uint32_t d2 = *reinterpret_cast<const uint32_t*>(&h);
#pragma unroll
                for (int j = 0; j < 4; ++j) cw[j] = c4;
#pragma unroll
                for (int j = 0; j < 8; ++j) dw[j] = d2;
            } else {
#pragma unroll
                for (int j = 0; j < 16; j += 2) {
                    const ulonglong2 kk = *reinterpret_cast<const ulonglong2*>(&s.key[key_index(xs + j, y)]);
                    const float z0 = kk.x ? fast_rcp(__uint_as_float((uint32_t)(kk.x >> 32))) : bg_z;
                    const float z1 = kk.y ? fast_rcp(__uint_as_float((uint32_t)(kk.y >> 32))) : bg_z;
                    const uint32_t c0 = kk.x ? (uint32_t)(kk.x & 0xff) : bg_cls, c1 = kk.y ? (uint32_t)(kk.y & 0xff) : bg_cls;
                    const __half2 h = __floats2half2_rn(z0, z1);
                    dw[j >> 1] = *reinterpret_cast<const uint32_t*>(&h);
                    if ((j & 3) == 0) cw[j >> 2] = c0 | (c1 << 8); else cw[j >> 2] |= (c0 << 16) | (c1 << 24);
                }
            }
            *reinterpret_cast<uint4*>(oc + o) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
            *reinterpret_cast<uint4*>(od + o) = make_uint4(dw[0], dw[1], dw[2], dw[3]);
            *reinterpret_cast<uint4*>(od + o + 8) = make_uint4(dw[4], dw[5], dw[6], dw[7]);
        } else {
            for (int j = 0; j < 16 && xs + j < t.tw; ++j) {
                const unsigned long long k = s.key[key_index(xs + j, y)];
                const float z = k ? fast_rcp(__uint_as_float((uint32_t)(k >> 32))) : bg_z;
                oc[o + j] = (uint8_t)(k ? (uint32_t)(k & 0xff) : bg_cls);
                od[o + j] = __half_as_ushort(__float2half_rn(z));
                if (o32) o32[o + j] = z;
            }
        }
    }
}

// Common prologue: tile geometry, camera, ray tables, frustum planes, cleared keys.
// Returns false when the ego is inactive (the tile is then all sky).
__device__ bool tile_prologue(TileSmem& s, TileCtx& t, const RenderParams& P, size_t& view, int& e, int& a) {
    const int tiles = P.tiles_x * P.tiles_y;
    const long long job = blockIdx.x;
    view = (size_t)(P.view_first + job / tiles);
    const int tile = (int)(job % tiles);
    const int k = (int)(view % P.K);
    a = (int)((view / P.K) % P.A);
    e = (int)(view / ((size_t)P.K * P.A));
    t.x0 = (tile % P.tiles_x) * TILE; t.y0 = (tile / P.tiles_x) * TILE;
    t.tw = min(TILE, P.W - t.x0); t.th = min(TILE, P.H - t.y0);
    t.w_near = P.w_near; t.w_far = P.w_far; t.near_z = P.near_z; t.far_z = P.far_z;
    t.med_cap = min(MCAP, P.med_cap); t.large_cap = min(LCAP, P.large_cap);
    const AgentGeom ego = P.agents[(size_t)e * P.A + a];
    if (threadIdx.x == 0) {
        make_camera(s.cam, ego, P.cam[k], P.W, P.H);
        s.n_large = 0; s.n_med = 0; s.n_leaf = 0; s.n_grp = 0; s.n_face = 0;
        s.touched[0] = 0u; s.touched[1] = 0u;
    }
    if (threadIdx.x < 16) s.cnt[threadIdx.x] = 0ull;
    if (threadIdx.x < 64) { s.bin_any[threadIdx.x] = 0ull; s.bin_full[threadIdx.x] = 0ull; }
    for (int i = threadIdx.x; i < TILE * TILE / 2; i += NTHREADS)
        reinterpret_cast<ulonglong2*>(s.key)[i] = make_ulonglong2(0ull, 0ull);
    __syncthreads();
    const Cam& c = s.cam;
    if (threadIdx.x < TILE) {
        const int i = threadIdx.x;
        s.ray_x[i] = __fdiv_rn(sub(add((float)(t.x0 + i), 0.5f), c.cx), c.focx);
        s.ray_y[i] = __fdiv_rn(sub(add((float)(t.y0 + i), 0.5f), c.cy), c.focy);
    }
    if (threadIdx.x >= 64 && threadIdx.x < 70) {
        // frustum planes n.(q - m_w) >= 0 with q = X - P_ego; unit normals, offset -n.m_w (+ near/far)
        const int p = threadIdx.x - 64;
        const float l = (float)t.x0 - c.cx, r = (float)(t.x0 + t.tw) - c.cx, u = (float)t.y0 - c.cy, d = (float)(t.y0 + t.th) - c.cy;
        float nx, ny, nz, off = 0.f, sx = 0.f, sy = 0.f, sz = 0.f;
        const float Rx = c.rx, Ry = c.ry, Dx = c.dx, Dy = c.dy, Dz = c.dz, Fx = c.fx_, Fy = c.fy_, Fz = c.fz_;
        switch (p) {
            case 0: nx = Fx; ny = Fy; nz = Fz; off = -P.near_z * 0.999f; break;                                       // z >= near
            case 1: nx = -Fx; ny = -Fy; nz = -Fz; off = P.far_z * 1.001f; break;                                      // z <= far
            case 2: nx = c.focx * Rx - l * Fx; ny = c.focx * Ry - l * Fy; nz = -l * Fz; sx = c.focx; sz = -l; break;  // x f >= z l
            case 3: nx = r * Fx - c.focx * Rx; ny = r * Fy - c.focx * Ry; nz = r * Fz; sx = -c.focx; sz = r; break;   // x f <= z r
            case 4: nx = c.focy * Dx - u * Fx; ny = c.focy * Dy - u * Fy; nz = c.focy * Dz - u * Fz; sy = c.focy; sz = -u; break;   // y f >= z u
            default: nx = d * Fx - c.focy * Dx; ny = d * Fy - c.focy * Dy; nz = d * Fz - c.focy * Dz; sy = -c.focy; sz = d; break;  // y f <= z d
        }
        const float inv = rsqrtf(nx * nx + ny * ny + nz * nz);
        nx *= inv; ny *= inv; nz *= inv;
        s.plane[p][0] = nx; s.plane[p][1] = ny; s.plane[p][2] = nz;
        s.plane[p][3] = off - (nx * c.mwx + ny * c.mwy + nz * c.mwz);
        if (p >= 2) {
            const float is = rsqrtf(sx * sx + sy * sy + sz * sz);
            s.side[p - 2][0] = sx * is; s.side[p - 2][1] = sy * is; s.side[p - 2][2] = sz * is; s.side[p - 2][3] = 0.f;
        }
    }
    __syncthreads();
    return ego.active != 0;
}

// ------------------------------------------------------------------------------------------------
// production kernel
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(NTHREADS, 4) render_kernel(const __grid_constant__ RenderParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TileSmem& s = *reinterpret_cast<TileSmem*>(smem_raw);
    TileCtx t;
    size_t view; int e, a;
    const bool count = P.counters != nullptr;
    long long c0 = count ? clock64() : 0;
    const bool ego_active = tile_prologue(s, t, P, view, e, a);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    Tally n = {0, 0, 0, 0, 0, 0, 0};
    int n_grp_tests = 0, n_leaf_tests = 0;
    long long c1 = 0, c2 = 0, c3 = 0, c4 = 0, c5 = 0;
    if (count) c1 = clock64();
    if (ego_active) {
        const MapInfo mi = P.maps[P.env_map[e]];
        // ---- (a)+(c) map: groups -> leaves -> primitives, set up as they survive
        for (uint32_t g0 = mi.group_begin; g0 < mi.group_end; g0 += GROUP_BATCH) {
            if (warp == 0) {
                const uint32_t g = g0 + lane;
                bool vis = false;
                if (lane < GROUP_BATCH && g < mi.group_end) { vis = box_visible(s, P.groups[g]); ++n_grp_tests; }
                const unsigned m = __ballot_sync(0xffffffffu, vis);
                if (vis) s.grp[__popc(m & ((1u << lane) - 1u))] = g;
                if (lane == 0) { s.n_grp = __popc(m); s.n_leaf = 0; }
            }
            __syncthreads();
            const int ng = s.n_grp;
            for (int i = warp; i < ng; i += NW) {
                const Node g = P.groups[s.grp[i]];
                bool vis = false;
                Node lf;
                if (lane < (int)g.count) { lf = P.leaves[g.first + lane]; vis = box_visible(s, lf); ++n_leaf_tests; }
                const unsigned m = __ballot_sync(0xffffffffu, vis);
                int base = 0;
                if (lane == 0 && m) base = atomicAdd(&s.n_leaf, __popc(m));
                base = __shfl_sync(0xffffffffu, base, 0);
                if (vis) s.leaf[base + __popc(m & ((1u << lane) - 1u))] = (lf.first << 4) | lf.count;
            }
            __syncthreads();
            const int nl = s.n_leaf;
            // LEAF_PRIMS threads per leaf, no barrier inside this loop
            for (int i = threadIdx.x; i < nl * LEAF_PRIMS; i += NTHREADS) {
                const uint32_t lf = s.leaf[i / LEAF_PRIMS];
                const uint32_t k = i % LEAF_PRIMS;
                if (k < (lf & 15u)) {
                    float v[12]; uint32_t key_lo, flags;
                    load_prim(P.prims + (lf >> 4) + k, v, key_lo, flags);
                    V3 V[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) V[j] = to_camera(s.cam, v[3 * j], v[3 * j + 1], v[3 * j + 2]);
                    process_prim(s, t, V, flags & 1u, flags, key_lo, n);
                }
            }
            __syncthreads();       // the leaf list is reused by the next batch and by the face items
        }
        if (count) c2 = clock64();
        // ---- (a)+(c) other agents: sphere cull per box, camera-facing faces become items
        const Cam& c = s.cam;
        for (int b0 = 0; b0 < P.A; b0 += LEAFCAP / 8) {
            for (int b = b0 + threadIdx.x; b < min(P.A, b0 + LEAFCAP / 8); b += NTHREADS) {
                if (b == a) continue;
                const AgentGeom g = P.agents[(size_t)e * P.A + b];
                if (!g.active) continue;
                const float hh = 0.5f * g.h;
                const V3 ctr = rotate_to_camera(c, sub(sub(g.x, c.px), c.mwx), sub(sub(g.y, c.py), c.mwy), sub(hh, c.mwz));
                const float rad = sqrtf(g.hl * g.hl + g.hw * g.hw + hh * hh) * 1.0001f + 1e-4f;
                bool vis = (ctr.z + rad >= t.near_z * 0.999f) && (ctr.z - rad <= t.far_z * 1.001f);
#pragma unroll
                for (int p = 0; p < 4; ++p)
                    vis = vis && (s.side[p][0] * ctr.x + s.side[p][1] * ctr.y + s.side[p][2] * ctr.z >= -rad);
                if (!vis) continue;
                // camera position in the box frame decides which faces can face the camera; near
                // the near plane (or inside the box) every face is kept
                uint32_t faces = 0x3fu;
                if (ctr.z - rad > t.near_z * 1.01f) {
                    const float dx = sub(c.mwx, sub(g.x, c.px)), dy = sub(c.mwy, sub(g.y, c.py));
                    const float u = g.c * dx + g.s * dy, v = g.c * dy - g.s * dx;
                    const float eps = 1e-4f * (1.f + fabsf(dx) + fabsf(dy));
                    faces = 0u;
                    if (u < -g.hl + eps) faces |= 1u;          // rear
                    if (u > g.hl - eps) faces |= 2u;           // front
                    if (v < -g.hw + eps) faces |= 4u;          // right
                    if (v > g.hw - eps) faces |= 8u;           // left
                    if (c.mwz < eps) faces |= 16u;             // bottom
                    if (c.mwz > g.h - eps) faces |= 32u;       // top
                }
                const int nf = __popc(faces);
                int slot = atomicAdd(&s.n_face, nf);
                for (; faces; faces &= faces - 1) s.face[slot++] = ((uint32_t)b << 3) | (uint32_t)(__ffs(faces) - 1);
            }
            __syncthreads();
            const int nf = s.n_face;
            for (int i = threadIdx.x; i < nf; i += NTHREADS) {
                const uint32_t it = s.face[i];
                const int b = (int)(it >> 3), f = (int)(it & 7u);
                const AgentGeom g = P.agents[(size_t)e * P.A + b];
                const uint32_t corners = face_corners(f);
                V3 V[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) V[k] = box_corner(c, g, (corners >> (4 * k)) & 7u);
                const uint32_t key_lo = ((0xFFFFFFu - (mi.n_tris + 12u * (uint32_t)b + 2u * (uint32_t)f)) << 8) | P.cls_agent;
                process_prim(s, t, V, true, face_flags(corners), key_lo, n);
            }
            __syncthreads();
            if (threadIdx.x == 0) s.n_face = 0;
            __syncthreads();
        }
        if (count) c3 = clock64();
        // ---- medium primitives (atomics) and binning of the large ones, then the block raster
        n.frags += raster_medium(s, t);
        bin_large(s, t);
        __syncthreads();
        if (threadIdx.x < 64 && s.bin_any[threadIdx.x]) mark_touched(s, 1ull << threadIdx.x);
        if (count) c4 = clock64();
        n.frags += raster_large(s, t);
    }
    __syncthreads();
    if (count) c5 = clock64();
    store_tile(s, t, P, view, ego_active);
    if (count) {
        atomicAdd(&s.cnt[1], (unsigned long long)n_grp_tests);
        atomicAdd(&s.cnt[2], (unsigned long long)n_leaf_tests);
        atomicAdd(&s.cnt[3], (unsigned long long)n.tested);
        atomicAdd(&s.cnt[4], (unsigned long long)n.setup);
        atomicAdd(&s.cnt[5], (unsigned long long)n.tiny);
        atomicAdd(&s.cnt[6], (unsigned long long)n.medium);
        atomicAdd(&s.cnt[7], (unsigned long long)n.large);
        atomicAdd(&s.cnt[8], (unsigned long long)n.fallback);
        atomicAdd(&s.cnt[9], (unsigned long long)n.frags);
        __syncthreads();
        if (threadIdx.x == 0) {
            const long long c6 = clock64();
            s.cnt[0] = 1;
            s.cnt[10] = (unsigned long long)(c1 - c0);
            if (ego_active) {
                s.cnt[11] = (unsigned long long)(c2 - c1); s.cnt[12] = (unsigned long long)(c3 - c2);
                s.cnt[13] = (unsigned long long)(c4 - c3); s.cnt[14] = (unsigned long long)(c5 - c4);
            }
            s.cnt[15] = (unsigned long long)(c6 - c5);
        }
        __syncthreads();
        if (threadIdx.x < 16 && s.cnt[threadIdx.x]) atomicAdd(&P.counters[threadIdx.x], s.cnt[threadIdx.x]);
    }
}

// ------------------------------------------------------------------------------------------------
// exhaustive kernel: every primitive of the map and every face of every other box against every
// pixel of the tile; no hierarchy, no frustum or pixel-box culling, no binning.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(NTHREADS) render_brute_kernel(const __grid_constant__ RenderParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TileSmem& s = *reinterpret_cast<TileSmem*>(smem_raw);
    TileCtx t;
    size_t view; int e, a;
    const bool ego_active = tile_prologue(s, t, P, view, e, a);
    if (ego_active) {
        const MapInfo mi = P.maps[P.env_map[e]];
        const uint32_t full = 0u | (0u << 8) | ((uint32_t)(t.tw - 1) << 16) | ((uint32_t)(t.th - 1) << 24);
        const uint32_t n_items = (mi.prim_end - mi.prim_begin) + 6u * (uint32_t)P.A;
        for (uint32_t i = threadIdx.x; i < n_items; i += NTHREADS) {
            V3 V[4]; bool quad; uint32_t flags, key_lo;
            if (i < mi.prim_end - mi.prim_begin) {
                float v[12];
                load_prim(P.prims + mi.prim_begin + i, v, key_lo, flags);
                quad = flags & 1u;
#pragma unroll
                for (int k = 0; k < 4; ++k) V[k] = to_camera(s.cam, v[3 * k], v[3 * k + 1], v[3 * k + 2]);
            } else {
                const uint32_t j = i - (mi.prim_end - mi.prim_begin);
                const int b = (int)(j / 6u), f = (int)(j % 6u);
                if (b == a) continue;
                const AgentGeom g = P.agents[(size_t)e * P.A + b];
                if (!g.active) continue;
                const uint32_t corners = face_corners(f);
#pragma unroll
                for (int k = 0; k < 4; ++k) V[k] = box_corner(s.cam, g, (corners >> (4 * k)) & 7u);
                quad = true; flags = face_flags(corners);
                key_lo = ((0xFFFFFFu - (mi.n_tris + 12u * (uint32_t)b + 2u * (uint32_t)f)) << 8) | P.cls_agent;
            }
            PrimEq q;
            if (!prim_equations(V, quad, flags, q)) continue;
            raster_in_thread(s, t, q, key_lo, full);
        }
    }
    __syncthreads();
    store_tile(s, t, P, view, ego_active);
}

// ------------------------------------------------------------------------------------------------
// host-side launchers (called from the C ABI)
// ------------------------------------------------------------------------------------------------
size_t render_smem_bytes() { return sizeof(TileSmem); }
int render_list_caps(int which) { return which == 0 ? MCAP : LCAP; }

cudaError_t configure_kernels() {
    cudaError_t err = cudaFuncSetAttribute(render_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TileSmem));
    if (err != cudaSuccess) return err;
    return cudaFuncSetAttribute(render_brute_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TileSmem));
}

cudaError_t launch_agents(int n, const float* poses, float* state, const float* actions, const float* dims,
                          const uint8_t* active, AgentGeom* out, uint32_t* status, float dt, float wheelbase,
                          float v_max, cudaStream_t stream) {
    if (n <= 0) return cudaSuccess;
    agent_kernel<<<(n + 127) / 128, 128, 0, stream>>>(n, poses, 3, state, actions, dims, active, out, status, dt,
                                                      wheelbase, v_max);
    return cudaGetLastError();
}

cudaError_t launch_render(const RenderParams& P, long long n_views, bool brute, cudaStream_t stream) {
    if (n_views <= 0) return cudaSuccess;
    const long long blocks = n_views * P.tiles_x * P.tiles_y;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (brute)
        render_brute_kernel<<<(unsigned)blocks, NTHREADS, sizeof(TileSmem), stream>>>(P);
    else
        render_kernel<<<(unsigned)blocks, NTHREADS, sizeof(TileSmem), stream>>>(P);
    return cudaGetLastError();
}

}  // namespace pic
