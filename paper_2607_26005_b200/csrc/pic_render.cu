// Production render kernels of the batched egocentric rasterizer (sm_100a).
//
// The z-buffer lives in shared memory as one 64-bit key per pixel,
//     key = float_bits(1/z) << 32 | (0xFFFFFF - primitive index) << 8 | class,
// so "nearest fragment wins, exact ties go to the lower index" is an unsigned max that does not
// depend on the order in which primitives arrive; 0 means "no fragment" (background).
//
// A unit of work is a tile: up to 64 x 64 pixels of one view.  Two kernels share the work.
//
// render_kernel (the fused kernel).  A CTA of 4 warps takes 4 consecutive tiles.
//   front   (a) cull, (c) set-up -- one warp per tile, warp-level synchronisation only.  The warp
//           tests the map's group boxes and the leaf boxes of the visible groups against the tile
//           frustum (a lane per box), culls the other agents' boxes as spheres and keeps their
//           camera-facing faces, then tests the candidates 32 at a time (camera-space vertices,
//           pixel box) and compacts the survivors with ballots.  Its lists live in the key buffer,
//           which is idle until the back end starts.  After one CTA barrier the survivors of the 4
//           tiles get consecutive ranges of a shared record pool and are set up, a lane per
//           survivor: 3-4 edge functions + 1/z plane in a 17-word record.
//   back    (b) raster, (c), (d) store -- after a second CTA barrier the 16 strips of 16 pixel rows
//           (4 per tile) are tasks that the warps draw from a counter.  A warp owns one strip of
//           keys (8 KB).  Per strip it looks at the tile's records 32 at a time (a lane each: does
//           the box reach the strip?), rasterizes primitives of <= 4 pixels from their lane with
//           atomic max, then walks the other hits together: a lane per pixel pair of a 16 x 4
//           pixel cell, plain loads and stores; boxes of >= 256 pixels first classify the strip's
//           16 cells (trivial reject / trivial accept / which edges still need testing) from the
//           same float32 edge functions.  The store converts keys to class u8 + depth binary16
//           with 128-bit stores, resets the keys it read, and writes 8 x 8 blocks that nothing
//           touched without reading keys.
//   Tiles whose lists overflow, or whose records do not fit the pool beside their fellows', are
//   appended to a list in device memory.
//
// cooperative_kernel.  One wave of CTAs walks that list; a whole CTA renders a tile in
// barrier-separated phases with per-round lists (any number of groups, boxes, survivors and
// records): the general path, and the one the fused kernel is checked against in the tests.
//
// Cameras (one 64-byte record per view) and per-camera ray / background tables are prepared by
// the agent and rig kernels, so the prologues are a few loads.
#include <cstddef>

#include "pic_device.cuh"

namespace pic {

// Profiling aid, compiled in only with -DPIC_PROFILE (never in the shipped library): bits 4-7 of the
// debug flags leave work out so that the cost of a phase can be timed by difference.  The images
// are then incomplete.
#ifdef PIC_PROFILE
#define PIC_STOP(P) (((P).debug_flags >> 4) & 15)
#else
#define PIC_STOP(P) 0
#endif

constexpr int NTHREADS = 128;
constexpr int NW = NTHREADS / 32;
constexpr int RCAP = 64;          // records (primitives rasterized by a warp) per tile
constexpr int REC = 20;           // words per record (17 used; 16-byte aligned for vector access)
constexpr int GROUP_BATCH = 16;   // groups examined per round
constexpr int LEAFCAP = GROUP_BATCH * GROUP_LEAVES;   // visible leaves per round
constexpr int BOX_ROUND = 64;     // boxes examined per round
constexpr int FACECAP = 6 * BOX_ROUND;
constexpr int SCAP = 128;         // candidates that survive the pixel-box test, per round
constexpr int TINY_MAX_PIXELS = 4;         // pixel centres in the box of a primitive rasterized by its own thread
static_assert(TINY_MAX_PIXELS == 4, "the strip back end enumerates the pixels of such a box for at most 4");
constexpr int CLASSIFY_MIN_PIXELS = 192;   // pixel boxes at least this large classify cells before rasterizing
#ifndef PIC_CLASSIFY_MIN
#define PIC_CLASSIFY_MIN 256
#endif
constexpr int CLASSIFY_MIN_STRIP = PIC_CLASSIFY_MIN;    // the same for the part of a box inside a 16-row strip

struct __align__(16) TileSmem {
    unsigned long long key[TILE * TILE];      // 32 KB, 16-byte chunks XOR-swizzled by row (key_index)
    float4 rec[RCAP * REC / 4];
    uint32_t leaf[LEAFCAP];                   // visible leaves of the round: first primitive << 4 | count
    uint32_t face[FACECAP];                   // box-face items of the round: agent << 3 | face
    uint2 surv[SCAP];                         // candidates whose pixel box holds a pixel centre: (item, box)
    float ray_x[TILE], ray_y[TILE];           // ray coordinates of the tile's pixel columns / rows
    float plane[6][4];                        // tile frustum, ego-relative world space, unit normals: n, offset
    float side[4][4];                         // the four side planes in camera space, unit normals
    Cam cam;
    int n_rec, n_leaf, n_face, n_surv;
    uint32_t touched[2];                      // 8x8 blocks that may hold a fragment (rows 0-3, rows 4-7)
};

// Keys are stored so that both access patterns spread over all banks.  A 16-byte chunk holds pixels
// (2c, 2c+1) of row y; its low three index bits are XORed with (y & 1) << 2 | (c >> 3).  Raster: a
// 16 x 4 cell is read a row (8 chunks of one 16-pixel column block) per quarter warp.  Store: 32
// consecutive lanes take 32 consecutive 16-pixel segments (two rows x four column blocks per quarter
// warp) and read chunk i of their segment together.
__device__ __forceinline__ int key_index(int x, int y) {
    const int c = x >> 1;
    return (y << 6) | (((c ^ (((y & 1) << 2) | (c >> 3))) << 1) | (x & 1));
}

// 256-bit store (sm_100): a lane's 16 depth values land in one fully written 32-byte sector.
__device__ __forceinline__ void store_256(void* p, const uint32_t (&w)[8]) {
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]),
                 "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                 : "memory");
}

// Bit mask of the 8x8 blocks touched by a pixel box (inclusive).
__device__ __forceinline__ unsigned long long block_mask(int bx0, int by0, int bx1, int by1) {
    const int c0 = bx0 >> 3, c1 = bx1 >> 3, r0 = by0 >> 3, r1 = by1 >> 3;
    const unsigned long long row = (unsigned long long)(((2u << c1) - (1u << c0)) & 0xffu);
    const unsigned long long rows = (0x0101010101010101ull >> (8 * (7 - (r1 - r0)))) << (8 * r0);
    return row * rows;
}

__device__ __forceinline__ void mark_touched(uint32_t* touched, unsigned long long m) {
    const uint32_t lo = (uint32_t)m, hi = (uint32_t)(m >> 32);
    if (lo & ~touched[0]) atomicOr(&touched[0], lo);
    if (hi & ~touched[1]) atomicOr(&touched[1], hi);
}

// Is the box [lo,hi] (world) possibly inside the tile frustum?  Conservative.
template <class S>
__device__ __forceinline__ bool box_visible(const S& s, const Node& b) {
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

template <class S>
__device__ __forceinline__ void put_fragment(S& s, int x, int y, uint32_t wbits, uint32_t key_lo) {
    const unsigned long long k = make_key(wbits, key_lo);
    unsigned long long* addr = &s.key[key_index(x, y)];
    atomicMax(addr, k);
}

// Rasterize a primitive from one thread: loop over its pixel box, atomic max per fragment.
template <class S>
__device__ __forceinline__ int raster_in_thread(S& s, uint32_t* touched, const TileCtx& t, const PrimEq& q, uint32_t key_lo, uint32_t box) {
    const int bx0 = box & 0xff, by0 = (box >> 8) & 0xff, bx1 = (box >> 16) & 0xff, by1 = box >> 24;
    int frags = 0;
    for (int y = by0; y <= by1; ++y) {
        const float ry = s.ray_y[y];
        for (int x = bx0; x <= bx1; ++x) {
            const uint32_t wb = fragment(q, s.ray_x[x], ry, t.w_near, t.w_far);
            if (wb) { put_fragment(s, x, y, wb, key_lo); ++frags; }
        }
    }
    if (frags) mark_touched(touched, block_mask(bx0, by0, bx1, by1));
    return frags;
}

// Plane p of the tile frustum, n.(q - m_w) >= 0 with q = X - P_ego (unit normals, offset -n.m_w
// plus near / far), and for p >= 2 the same side plane in camera space.
template <class S>
__device__ __forceinline__ void tile_planes(S& s, int p, const Cam& c, const TileCtx& t) {
    const float l = (float)t.x0 - c.cx, r = (float)(t.x0 + t.tw) - c.cx, u = (float)t.y0 - c.cy, d = (float)(t.y0 + t.th) - c.cy;
    float nx, ny, nz, off = 0.f, sx = 0.f, sy = 0.f, sz = 0.f;
    const float Rx = c.rx, Ry = c.ry, Dx = c.dx, Dy = c.dy, Dz = c.dz, Fx = c.fx_, Fy = c.fy_, Fz = c.fz_;
    switch (p) {
        case 0: nx = Fx; ny = Fy; nz = Fz; off = -t.near_z * 0.999f; break;                                       // z >= near
        case 1: nx = -Fx; ny = -Fy; nz = -Fz; off = t.far_z * 1.001f; break;                                      // z <= far
        case 2: nx = c.focx * Rx - l * Fx; ny = c.focx * Ry - l * Fy; nz = -l * Fz; sx = c.focx; sz = -l; break;  // x f >= z l
        case 3: nx = r * Fx - c.focx * Rx; ny = r * Fy - c.focx * Ry; nz = r * Fz; sx = -c.focx; sz = r; break;   // x f <= z r
        case 4: nx = c.focy * Dx - u * Fx; ny = c.focy * Dy - u * Fy; nz = c.focy * Dz - u * Fz; sy = c.focy; sz = -u; break;
        default: nx = d * Fx - c.focy * Dx; ny = d * Fy - c.focy * Dy; nz = d * Fz - c.focy * Dz; sy = -c.focy; sz = d; break;
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

// Which faces of another agent's box can reach the tile: 0 if its bounding sphere misses the
// frustum, else the faces that can face the camera (all six near the near plane or inside the box).
template <class S>
__device__ __forceinline__ uint32_t box_faces(const S& s, const Cam& c, const TileCtx& t, const AgentGeom& g) {
    const float hh = 0.5f * g.h;
    const V3 ctr = rotate_to_camera(c, sub(sub(g.x, c.px), c.mwx), sub(sub(g.y, c.py), c.mwy), sub(hh, c.mwz));
    const float rad = sqrtf(g.hl * g.hl + g.hw * g.hw + hh * hh) * 1.0001f + 1e-4f;
    bool vis = (ctr.z + rad >= t.near_z * 0.999f) && (ctr.z - rad <= t.far_z * 1.001f);
#pragma unroll
    for (int p = 0; p < 4; ++p)
        vis = vis && (s.side[p][0] * ctr.x + s.side[p][1] * ctr.y + s.side[p][2] * ctr.z >= -rad);
    if (!vis) return 0u;
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
    return faces;
}

// Work counters of a thread; the production kernel is compiled with NoTally, where they vanish.
struct Tally { int grp, leaf, tested, setup, tiny, recs, fallback, classified, cells, jobs, coop; };
struct NoCount {
    __device__ __forceinline__ NoCount& operator++() { return *this; }
    __device__ __forceinline__ NoCount& operator=(int) { return *this; }
};
__device__ __forceinline__ int tally_value(int v) { return v; }
__device__ __forceinline__ int tally_value(const NoCount&) { return 0; }
struct NoTally { NoCount grp, leaf, tested, setup, tiny, recs, fallback, classified, cells, jobs, coop; };

// Cooperative kernel, phase 2b body: set a surviving primitive up, rasterize it (tiny) or leave a record.
template <class TL>
__device__ __forceinline__ void setup_prim(TileSmem& s, const TileCtx& t, const V3 (&V)[4], bool quad, uint32_t flags,
                                           const V3 Pn, uint32_t key_lo, uint32_t box, int rec_cap, TL& n) {
    PrimEq q;
    if (!prim_equations(V, quad, flags, Pn, q)) return;
    ++n.setup;
    const int bx0 = box & 0xff, by0 = (box >> 8) & 0xff, bx1 = (box >> 16) & 0xff, by1 = box >> 24;
    if ((bx1 - bx0 + 1) * (by1 - by0 + 1) > TINY_MAX_PIXELS) {
        const int slot = atomicAdd(&s.n_rec, 1);
        if (slot < rec_cap) {
            float4* r = &s.rec[slot * (REC / 4)];
            r[0] = make_float4(q.nx[0], q.nx[1], q.nx[2], q.nx[3]);
            r[1] = make_float4(q.ny[0], q.ny[1], q.ny[2], q.ny[3]);
            r[2] = make_float4(q.nz[0], q.nz[1], q.nz[2], q.nz[3]);
            r[3] = make_float4(q.wx, q.wy, q.wz, __uint_as_float(key_lo));
            // the pixel box needs 6 bits per coordinate; the top-left bits ride along
            r[4].x = __uint_as_float((uint32_t)bx0 | ((uint32_t)by0 << 6) | ((uint32_t)bx1 << 12) | ((uint32_t)by1 << 18) | (q.tl << 24));
            ++n.recs;
            return;
        }
        ++n.fallback;          // list full: correct but slow
    } else {
        ++n.tiny;
    }
    raster_in_thread(s, s.touched, t, q, key_lo, box);
}

// Candidate `i` of the round: a primitive of a visible leaf or a box-face item, in camera space.
template <class S>
__device__ __forceinline__ bool fetch_candidate(const S& s, const RenderParams& P, int i, int nl, int e, uint32_t n_map_tris,
                                                V3 (&V)[4], V3& Pn, uint32_t& key_lo, uint32_t& flags, bool want_plane) {
    const Cam& c = s.cam;
    if (i < nl * LEAF_PRIMS) {
        const uint32_t lf = s.leaf[i / LEAF_PRIMS];
        const uint32_t j = i % LEAF_PRIMS;
        if (j >= (lf & 15u)) return false;
        float v[12], vis_cos;
        load_prim(P.prims + (lf >> 4) + j, v, key_lo, flags, vis_cos);
#pragma unroll
        for (int q = 0; q < 4; ++q) V[q] = to_camera(c, v[3 * q], v[3 * q + 1], v[3 * q + 2]);
        if (want_plane) Pn = limit_angular_range(V, plane_normal_world(c, v, flags & 1u), vis_cos);
    } else {
        const uint32_t it = s.face[i - nl * LEAF_PRIMS];
        const int b = (int)(it >> 3), f = (int)(it & 7u);
        const AgentGeom g = P.agents[(size_t)e * P.A + b];
        const uint32_t corners = face_corners(f);
#pragma unroll
        for (int q = 0; q < 4; ++q) V[q] = box_corner(c, g, (corners >> (4 * q)) & 7u);
        key_lo = ((0xFFFFFFu - (n_map_tris + 12u * (uint32_t)b + 2u * (uint32_t)f)) << 8) | agent_box_class(g);
        flags = face_flags(corners);
        if (want_plane) Pn = plane_normal(V, true);
    }
    return true;
}

// The top-left rule "e > 0 || (e == 0 && the edge owns its zeros)" as one comparison e > thr:
// thr is 0 or the smallest negative subnormal -- nothing lies between the two, and neither fma nor
// the comparison flushes subnormals.
__device__ __forceinline__ void edge_thresholds(uint32_t tl, float (&thr)[4]) {
#pragma unroll
    for (int e = 0; e < 4; ++e) thr[e] = __int_as_float(((tl >> e) & 1u) ? (int)0x80000001u : 0);
}

// One 16 x 4 cell at (xx, yy): every lane tests its two pixels and updates their keys with plain
// loads and stores -- the rows of a cell belong to exactly one warp (its strip in the fused kernel,
// its bands in the cooperative kernel).  `need`: the edges
// that still have to be tested on this cell (0: the cell is known to be covered and in depth
// range; the range test rides on the edge tests).  Returns whether any lane produced a fragment.
template <class S>
__device__ __forceinline__ bool raster_cell(S& s, const TileCtx& t, const PrimEq& q, const float (&thr)[4], uint32_t key_lo, int xx, int yy,
                                            uint32_t need, int lane) {
    const int x = xx + (lane & 7) * 2, y = yy + (lane >> 3);
    const float rx0 = s.ray_x[x], rx1 = s.ray_x[x + 1], ry = s.ray_y[y];
    const float wt = fm(q.wy, ry, q.wz);
    const float w0 = fm(q.wx, rx0, wt), w1 = fm(q.wx, rx1, wt);
    bool in0 = true, in1 = true;
    if (need) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if ((need >> e) & 1u) {          // warp-uniform: edges known to be positive on the whole cell are skipped
                const float te = fm(q.ny[e], ry, q.nz[e]);
                const float e0 = fm(q.nx[e], rx0, te), e1 = fm(q.nx[e], rx1, te);
                in0 = in0 && (e0 > thr[e]);
                in1 = in1 && (e1 > thr[e]);
            }
        }
        in0 = in0 && (w0 >= t.w_far) && (w0 <= t.w_near);
        in1 = in1 && (w1 >= t.w_far) && (w1 <= t.w_near);
    }
    {
        ulonglong2* kp = reinterpret_cast<ulonglong2*>(&s.key[key_index(x, y)]);
        ulonglong2 kk = *kp;
        const unsigned long long k0 = make_key(__float_as_uint(w0), key_lo), k1 = make_key(__float_as_uint(w1), key_lo);
        const bool up0 = in0 && k0 > kk.x, up1 = in1 && k1 > kk.y;
        if (up0) kk.x = k0;
        if (up1) kk.y = k1;
        if (up0 || up1) *kp = kk;
    }
    return __any_sync(0xffffffffu, in0 || in1);
}

// Cooperative kernel, phase 3: every warp walks all records but rasterizes only the bands (4 pixel rows) it owns --
// band b belongs to warp b % NW -- so keys are updated without atomics and the bands of a large
// primitive are shared out evenly.
template <class S, class TL>
__device__ __forceinline__ void raster_records(S& s, const float4* rec, uint32_t* touched_out, const TileCtx& t, int n_rec, bool classify, TL& n) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned long long touched = 0ull;     // 8x8 blocks
    for (int p = 0; p < n_rec; ++p) {
        const float4* r = &rec[p * (REC / 4)];
        const uint32_t bw = __float_as_uint(r[4].x);
        if (bw >> 28) continue;                  // rasterized by its own thread, or degenerate
        const int bx0 = bw & 63, by0 = (bw >> 6) & 63, bx1 = (bw >> 12) & 63, by1 = (bw >> 18) & 63;
        // first band of this warp at or after the box's first band
        const int band0 = by0 >> 2, band1 = by1 >> 2;
        int first = band0 + ((warp - band0) & (NW - 1));
        if (first > band1) continue;
        PrimEq q;
        const float4 r0 = r[0], r1 = r[1], r2 = r[2], r3 = r[3];
        q.nx[0] = r0.x; q.nx[1] = r0.y; q.nx[2] = r0.z; q.nx[3] = r0.w;
        q.ny[0] = r1.x; q.ny[1] = r1.y; q.ny[2] = r1.z; q.ny[3] = r1.w;
        q.nz[0] = r2.x; q.nz[1] = r2.y; q.nz[2] = r2.z; q.nz[3] = r2.w;
        q.wx = r3.x; q.wy = r3.y; q.wz = r3.z;
        const uint32_t key_lo = __float_as_uint(r3.w);
        q.tl = (bw >> 24) & 15u;
        float thr[4];
        edge_thresholds(q.tl, thr);
        if (classify && (bx1 - bx0 + 1) * (by1 - by0 + 1) >= CLASSIFY_MIN_PIXELS) {
            // (b) lanes 0..15 classify this warp's 16 cells: reject / partly covered / inside
            if (warp == 0) ++n.classified;
            const int band = (lane >> 2) * NW + warp, col = lane & 3;
            const int xa = col * 16, xb = xa + 15, ya = band * 4, yb = ya + 3;
            bool reject = lane >= 16 || xb < bx0 || xa > bx1 || yb < by0 || ya > by1;
            uint32_t need = 0u;
            if (!reject) {
                const float rxa = s.ray_x[xa], rxb = s.ray_x[xb], rya = s.ray_y[ya], ryb = s.ray_y[yb];   // rxa < rxb, rya < ryb
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    // fma is monotone in each argument, so the cell's extreme values are at its corners
                    const float ta = fm(q.ny[e], rya, q.nz[e]), tb = fm(q.ny[e], ryb, q.nz[e]);
                    const float emax = fm(q.nx[e], q.nx[e] >= 0.f ? rxb : rxa, fmaxf(ta, tb));
                    const float emin = fm(q.nx[e], q.nx[e] >= 0.f ? rxa : rxb, fminf(ta, tb));
                    reject = reject || (emax < 0.f);
                    if (!(emin > 0.f)) need |= 1u << e;
                }
                const float wa = fm(q.wy, rya, q.wz), wb = fm(q.wy, ryb, q.wz);
                const float wmax = fm(q.wx, q.wx >= 0.f ? rxb : rxa, fmaxf(wa, wb));
                const float wmin = fm(q.wx, q.wx >= 0.f ? rxa : rxb, fminf(wa, wb));
                reject = reject || (wmax < t.w_far) || (wmin > t.w_near);
                // the depth range test rides on the edge tests: if it is still needed, so is one edge
                if (need == 0u && !((wmin >= t.w_far) && (wmax <= t.w_near))) need = 1u;
            }
            for (unsigned m = __ballot_sync(0xffffffffu, !reject); m; m &= m - 1) {
                const int cell = __ffs(m) - 1;
                const int xx = (cell & 3) * 16, yy = ((cell >> 2) * NW + warp) * 4;
                const uint32_t need_c = __shfl_sync(0xffffffffu, need, cell);
                ++n.cells;
                if (raster_cell(s, t, q, thr, key_lo, xx, yy, need_c, lane)) touched |= 3ull << ((yy >> 3) * 8 + (xx >> 3));
            }
        } else {
            for (int band = first; band <= band1; band += NW)
                for (int xx = bx0 & ~15; xx <= bx1; xx += 16) {
                    ++n.cells;
                    if (raster_cell(s, t, q, thr, key_lo, xx, band * 4, 0xFu, lane)) touched |= 3ull << ((band >> 1) * 8 + (xx >> 3));
                }
        }
    }
    if (lane == 0 && touched) mark_touched(touched_out, touched);
}

// (d) keys -> class / depth images.  `touched`: the 8x8 blocks that may hold a fragment; with
// `clear`, the keys that were read are reset to "no fragment" for the next tile.
// FULL: the caller guarantees full tiles of an image whose rows allow 128-bit stores and no float32
// depth image, so that only the vector path is compiled in.
template <bool FULL = false, class S>
__device__ __forceinline__ void store_tile(S& s, const TileCtx& t, const RenderParams& P, size_t view, int k, bool ego_active,
                                           unsigned long long touched, bool clear, int tid = threadIdx.x, int nthr = NTHREADS,
                                           uint32_t n_map_tris = 0u) {
    const size_t img = (size_t)P.H * P.W;
    uint32_t* occ = (!FULL && P.occlusion) ? P.occlusion + view * (size_t)P.A * 2u : nullptr;   // visible-pixel counts of this view
    uint8_t* oc = P.out_class + view * img;
    uint16_t* od = P.out_depth + view * img;
    float* o32 = P.out_depth32 ? P.out_depth32 + view * img : nullptr;
    const bool vec_ok = FULL || ((P.W % 16 == 0) && o32 == nullptr);
    const int segs_per_row = FULL ? TILE / 16 : (t.tw + 15) >> 4;
    const int n_seg = t.th * segs_per_row;
    // consecutive threads take consecutive 16-pixel segments of a row, then the next row: a warp's
    // class stores cover 512 contiguous bytes of a 64-pixel-wide image, its depth stores 1 KB
    for (int seg = tid; seg < n_seg; seg += nthr) {
        const int y = FULL ? seg >> 2 : seg / segs_per_row;
        const int xs = (seg - y * segs_per_row) * 16;
        uint32_t bg_cls = P.cls_sky;
        float bg_z = P.far_z;
        if (ego_active) { bg_cls = __ldg(P.rig.bg_cls + (size_t)k * P.H + t.y0 + y); bg_z = __ldg(P.rig.bg_z + (size_t)k * P.H + t.y0 + y); }
        const size_t o = (size_t)(t.y0 + y) * P.W + t.x0 + xs;
        const bool empty = ((touched >> ((y >> 3) * 8 + (xs >> 3))) & 3ull) == 0ull;   // both blocks of the segment
        if (FULL || (vec_ok && xs + 16 <= t.tw)) {
            uint32_t cw[4], dw[8];
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
                    ulonglong2* kp = reinterpret_cast<ulonglong2*>(&s.key[key_index(xs + j, y)]);
                    const ulonglong2 kk = *kp;
                    if (clear) *kp = make_ulonglong2(0ull, 0ull);
                    if (occ) { count_visible(occ, kk.x, n_map_tris); count_visible(occ, kk.y, n_map_tris); }
                    const float z0 = kk.x ? fast_rcp(__uint_as_float((uint32_t)(kk.x >> 32))) : bg_z;
                    const float z1 = kk.y ? fast_rcp(__uint_as_float((uint32_t)(kk.y >> 32))) : bg_z;
                    const uint32_t c0 = kk.x ? (uint32_t)(kk.x & 0xff) : bg_cls, c1 = kk.y ? (uint32_t)(kk.y & 0xff) : bg_cls;
                    const __half2 h = __floats2half2_rn(z0, z1);
                    dw[j >> 1] = *reinterpret_cast<const uint32_t*>(&h);
                    if ((j & 3) == 0) cw[j >> 2] = c0 | (c1 << 8); else cw[j >> 2] |= (c0 << 16) | (c1 << 24);
                }
            }
#ifdef PIC_PROFILE
            if (PIC_STOP(P) == 6 && !(P.debug_flags & 0x10000)) continue;
#endif
            *reinterpret_cast<uint4*>(oc + o) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
            if (FULL) {
                store_256(od + o, dw);
            } else {
                *reinterpret_cast<uint4*>(od + o) = make_uint4(dw[0], dw[1], dw[2], dw[3]);
                *reinterpret_cast<uint4*>(od + o + 8) = make_uint4(dw[4], dw[5], dw[6], dw[7]);
            }
        } else {
            for (int j = 0; j < 16 && xs + j < t.tw; ++j) {
                const unsigned long long key = empty ? 0ull : s.key[key_index(xs + j, y)];
                if (clear && !empty) s.key[key_index(xs + j, y)] = 0ull;
                if (occ) count_visible(occ, key, n_map_tris);
                const float z = key ? fast_rcp(__uint_as_float((uint32_t)(key >> 32))) : bg_z;
                oc[o + j] = (uint8_t)(key ? (uint32_t)(key & 0xff) : bg_cls);
                od[o + j] = __half_as_ushort(__float2half_rn(z));
                if (o32) o32[o + j] = z;
            }
        }
    }
}

// One unit of work: a tile of a view.
struct Job {
    int tile, k, a, e;
    size_t view;
    TileCtx t;
};

// Job `id` of the launch: tiles of a view are consecutive, views follow P.view_first.
__device__ __forceinline__ Job decode_job(const RenderParams& P, unsigned id) {
    const unsigned tiles = (unsigned)(P.tiles_x * P.tiles_y);
    const unsigned vrel = id / tiles;
    const unsigned long long v = (unsigned long long)P.view_first + vrel;
    Job j;
    j.tile = (int)(id - vrel * tiles);
    j.view = (size_t)v;
    const unsigned va = (unsigned)(v / (unsigned)P.K);        // E * A * K < 2^31 (checked by the launcher)
    j.k = (int)((unsigned)v - va * (unsigned)P.K);
    j.e = (int)(va / (unsigned)P.A);
    j.a = (int)(va - (unsigned)j.e * (unsigned)P.A);
    j.t.x0 = (j.tile % P.tiles_x) * TILE; j.t.y0 = (j.tile / P.tiles_x) * TILE;
    j.t.tw = min(TILE, P.W - j.t.x0); j.t.th = min(TILE, P.H - j.t.y0);
    j.t.w_near = P.w_near; j.t.w_far = P.w_far; j.t.near_z = P.near_z; j.t.far_z = P.far_z;
    return j;
}

// Ray coordinates of tile column / row i (threads 0..63 of a pass call this with i = 0..63).
// Columns / rows past the image edge (ragged tiles) continue the same formula, so the tables
// stay monotone for the cell classification.
template <class S>
__device__ __forceinline__ void load_rays(S& s, const RenderParams& P, const Job& j, int i) {
    const CamConst& ck = P.cam[j.k];
    s.ray_x[i] = (j.t.x0 + i < P.W) ? __ldg(P.rig.ray_x + (size_t)j.k * P.W + j.t.x0 + i)
                                    : __fdiv_rn(sub(add((float)(j.t.x0 + i), 0.5f), 0.5f * (float)P.W), ck.fx);
    s.ray_y[i] = (j.t.y0 + i < P.H) ? __ldg(P.rig.ray_y + (size_t)j.k * P.H + j.t.y0 + i)
                                    : __fdiv_rn(sub(add((float)(j.t.y0 + i), 0.5f), 0.5f * (float)P.H), ck.fy);
}

// A whole tile rendered by the CTA in barrier-separated phases with per-round lists: any number of
// groups, boxes, survivors and records.  It serves the tiles that the fused kernel leaves out.
template <class TL, bool FULL>
__device__ __forceinline__ void cooperative_job(TileSmem& s, const RenderParams& P, unsigned job_id, TL& n) {
    const Job job = decode_job(P, job_id);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool classify = !(P.debug_flags & 1);
    const int rec_cap = (P.debug_flags & 2) ? 2 : RCAP;
    const int stop = PIC_STOP(P);
    const int k = job.k, a = job.a, e = job.e;
    const size_t view = job.view;
    const TileCtx t = job.t;
    const bool ego_active = P.agents[(size_t)e * P.A + a].active != 0;
    // issued now so that their latency overlaps the prologue: the map of this environment, the
    // group box this lane tests first, and the background of the two rows this thread stores
    const MapInfo mi = P.env_maps[e];
    Node gn0;
    gn0.first = 0; gn0.count = 0;
    if (lane < GROUP_BATCH && mi.group_begin + lane < mi.group_end) gn0 = P.groups[mi.group_begin + lane];

    // ---- prologue: camera, ray tables, frustum planes, cleared keys
    if (threadIdx.x < 7) {
        Cam c;
        load_camera(c, P.cams[view], P.cam[k], P.W, P.H);
        if (threadIdx.x == 6) {
            s.cam = c;
            s.n_rec = 0; s.n_leaf = 0; s.n_face = 0; s.n_surv = 0;
            s.touched[0] = 0u; s.touched[1] = 0u;
        } else {
            tile_planes(s, threadIdx.x, c, t);
        }
    } else if (threadIdx.x >= 64) {
        load_rays(s, P, job, threadIdx.x - 64);
    }
#pragma unroll
    for (int i = 0; i < TILE * TILE / 2 / NTHREADS; ++i)
        reinterpret_cast<ulonglong2*>(s.key)[i * NTHREADS + threadIdx.x] = make_ulonglong2(0ull, 0ull);
    __syncthreads();

    if (ego_active && stop != 1) {
        const Cam& c = s.cam;
        const uint32_t n_groups = mi.group_end - mi.group_begin;
        const int n_rounds = max((int)((n_groups + GROUP_BATCH - 1) / GROUP_BATCH), (P.A + BOX_ROUND - 1) / BOX_ROUND);
        for (int round = 0; round < n_rounds; ++round) {
            // ---- phase 1 (a): hierarchy and boxes of this round
            const uint32_t g0 = mi.group_begin + (uint32_t)round * GROUP_BATCH;
            if (g0 < mi.group_end) {
                const uint32_t g = g0 + lane;
                bool vis = false;
                Node gn;
                if (lane < GROUP_BATCH && g < mi.group_end) { gn = (round == 0) ? gn0 : P.groups[g]; vis = box_visible(s, gn); if (warp == 0) ++n.grp; }
                unsigned gm = __ballot_sync(0xffffffffu, vis);
                // warp w takes the visible groups w, w + NW, ...
                for (int i = 0; gm; gm &= gm - 1, ++i) {
                    if ((i & (NW - 1)) != warp) continue;
                    const int src = __ffs(gm) - 1;
                    const uint32_t first = __shfl_sync(0xffffffffu, gn.first, src);
                    const uint32_t cnt = __shfl_sync(0xffffffffu, gn.count, src);
                    bool lvis = false;
                    Node lf;
                    if (lane < (int)cnt) { lf = P.leaves[first + lane]; lvis = box_visible(s, lf); ++n.leaf; }
                    const unsigned lm = __ballot_sync(0xffffffffu, lvis);
                    int base = 0;
                    if (lane == 0 && lm) base = atomicAdd(&s.n_leaf, __popc(lm));
                    base = __shfl_sync(0xffffffffu, base, 0);
                    if (lvis) s.leaf[base + __popc(lm & ((1u << lane) - 1u))] = (lf.first << 4) | lf.count;
                }
            }
            // boxes are taken from the last thread down: the first warps are busier with the visible groups
            for (int b = round * BOX_ROUND + (NTHREADS - 1 - (int)threadIdx.x); b < min(P.A, (round + 1) * BOX_ROUND); b += NTHREADS) {
                if (b == a) continue;
                const AgentGeom g = P.agents[(size_t)e * P.A + b];
                if (!g.active) continue;
                uint32_t faces = box_faces(s, c, t, g);
                if (!faces) continue;
                int slot = atomicAdd(&s.n_face, __popc(faces));
                for (; faces; faces &= faces - 1) s.face[slot++] = ((uint32_t)b << 3) | (uint32_t)(__ffs(faces) - 1);
            }
            __syncthreads();
            // ---- phase 2a (a): one thread per candidate: camera space, pixel box; survivors are compacted
            const int nl = s.n_leaf, nf = s.n_face;
            const int n_items = (stop == 2) ? 0 : nl * LEAF_PRIMS + nf;
            for (int i0 = 0; i0 < n_items; i0 += NTHREADS) {
                const int i = i0 + threadIdx.x;
                V3 V[4], Pn;
                uint32_t key_lo, flags, box = 0;
                bool keep = false;
                if (i < n_items && fetch_candidate(s, P, i, nl, e, mi.n_tris, V, Pn, key_lo, flags, false)) {
                    ++n.tested;
                    keep = pixel_box(c, t, V, box);
                }
                const unsigned m = __ballot_sync(0xffffffffu, keep);
                int base = 0;
                if (lane == 0 && m) base = atomicAdd(&s.n_surv, __popc(m));
                base = __shfl_sync(0xffffffffu, base, 0);
                if (keep) {
                    const int slot = base + __popc(m & ((1u << lane) - 1u));
                    if (slot < SCAP) s.surv[slot] = make_uint2((uint32_t)i, box);
                    else {                                                                  // list full (rare)
                        fetch_candidate(s, P, i, nl, e, mi.n_tris, V, Pn, key_lo, flags, true);
                        setup_prim(s, t, V, flags & 1u, flags, Pn, key_lo, box, rec_cap, n);
                    }
                }
            }
            __syncthreads();
            // ---- phase 2b (c): one thread per survivor: edge functions, 1/z plane, tiny raster or record
            const int ns = (stop == 3) ? 0 : min(s.n_surv, SCAP);
            for (int j = threadIdx.x; j < ns; j += NTHREADS) {
                const uint2 sv = s.surv[j];
                V3 V[4], Pn;
                uint32_t key_lo, flags;
                fetch_candidate(s, P, (int)sv.x, nl, e, mi.n_tris, V, Pn, key_lo, flags, true);
                setup_prim(s, t, V, flags & 1u, flags, Pn, key_lo, sv.y, rec_cap, n);
            }
            __syncthreads();
            if (round + 1 < n_rounds) {
                // the lists are reused by the next round; records are rasterized now if they might overflow
                const int n_rec = min(s.n_rec, rec_cap);
                if (n_rec > rec_cap / 2) raster_records(s, s.rec, s.touched, t, n_rec, classify, n);
                __syncthreads();
                if (threadIdx.x == 0) { s.n_leaf = 0; s.n_face = 0; s.n_surv = 0; if (n_rec > rec_cap / 2) s.n_rec = 0; }
                __syncthreads();
            }
        }
        // ---- phase 3 (b)+(c): one warp per record
        if (stop == 0 || stop > 5) raster_records(s, s.rec, s.touched, t, min(s.n_rec, rec_cap), classify, n);
        if (stop == 5 && threadIdx.x == 0) { s.touched[0] = 0xffffffffu; s.touched[1] = 0xffffffffu; }
        __syncthreads();
    }
    // ---- phase 4 (d)
    store_tile<FULL>(s, t, P, view, k, ego_active, ((unsigned long long)s.touched[1] << 32) | s.touched[0], false, threadIdx.x, NTHREADS, mi.n_tris);
    if (threadIdx.x == 0) { ++n.jobs; ++n.coop; }
}

// Adds the CTA's tallies to the optional counters: [0] tiles, [1..9] group tests, leaf tests,
// candidates tested, set up, rasterized by their thread, records, record-list overflows, records
// classified per cell, cells visited, [10] tiles rendered by cooperative_job.
__device__ __forceinline__ void flush_counters(const RenderParams&, const NoTally&) {}
__device__ __forceinline__ void flush_counters(const RenderParams& P, const Tally& n) {
    const int lane = threadIdx.x & 31;
    const int vals[11] = {n.jobs, n.grp, n.leaf, n.tested, n.setup, n.tiny, n.recs, n.fallback, n.classified, n.cells, n.coop};
#pragma unroll
    for (int i = 0; i < 11; ++i) {
        // classified / cells are counted by every lane of a warp alike
        const int v = ((i == 8 || i == 9) && lane != 0) ? 0 : vals[i];
        const int sum = __reduce_add_sync(0xffffffffu, v);
        if (lane == 0 && sum) atomicAdd(&P.counters[i], (unsigned long long)sum);
    }
}

// ---------------------------------------------------------------------------------------------
// Fused kernel: a CTA takes NW consecutive tiles (see the head of this file).
//
//   front   warp w culls tile w on its own (hierarchy, boxes, candidate tests), with warp-level
//           synchronisation only and its lists in its (still unused) strip of keys; after a CTA
//           barrier the survivors of the NW tiles get consecutive ranges of one record pool and
//           are set up, one lane per survivor.  Dense passes.
//   back    after a second CTA barrier, 16-row strips are tasks drawn from a counter: a warp
//           rasterizes a strip of some tile into its own strip of keys and stores it (back_strip).
//   rest    tiles whose lists or records did not fit are appended to the cooperative kernel's list.
// ---------------------------------------------------------------------------------------------
constexpr int POOL = 128;         // records shared by the NW tiles of a CTA
constexpr int STRIP = 16;         // pixel rows a warp rasterizes at a time
constexpr int STRIP_KEYS = TILE * STRIP;
constexpr int W_FACE = 384;        // box-face items of a tile in the cull kernel
// Survivor buffer, SURV_STRIDE uint2 per tile: a 16-byte head (counts; work counts), then W_SURV
// entries (id, pixel box).  Survivors whose pixel box holds more than TINY_MAX_PIXELS pixel centres
// fill the list from the front, the others from the back; head.x = front count | back count << 16,
// or all ones if a list overflowed.
constexpr int SURV_STRIDE = 256;
constexpr int W_SURV = SURV_STRIDE - 2;
constexpr uint32_t SURV_OVERFLOW = 0xffffffffu;
constexpr uint32_t SURV_FACE = 0x80000000u;   // survivor id: index into grid_prims, or SURV_FACE | agent << 3 | face
constexpr uint32_t REC_TINY = 1u << 28, REC_DEAD = 1u << 29;   // flags in the box word of a record
constexpr uint32_t REC_INRANGE = 1u << 30;   // every covered pixel is within [near, far]: no per-pixel range test

constexpr int W_LARGE = 64;       // visible leaves of the large-primitive list
struct __align__(16) FrontLists {
    float plane[6][4];                        // (read as float4: kept first, 16-byte aligned)
    float side[4][4];
    Cam cam;
    float seg[10][6];                         // footprint segments: x, y, dx, dy, 1 / dy, unused
    float pt[5][2];                           // footprint corners (ego-relative xy): apex, four far corners
    uint32_t face[W_FACE];                    // agent << 3 | face
    uint32_t lleaf[W_LARGE];                  // visible large-primitive leaves: first << 3 | count
    uint32_t row_first[32];                   // grid rows of a pass: first entry of the row's range in cell_prims
    uint32_t row_off[33];                     //   and the number of candidates before the row (the total at [32])
    int n_face;
};
static_assert(offsetof(FrontLists, plane) % 16 == 0 && offsetof(FrontLists, side) % 16 == 0, "planes are read with 128-bit loads");

struct __align__(16) FusedSmem {
    unsigned long long key[NW][STRIP_KEYS];   // warp w's strip of keys; during the front end, its FrontLists
    float4 pool[POOL * REC / 4];
    float ray_x[NW][TILE], ray_y[NW][STRIP];  // ray tables of the strip a warp works on
    int n_surv[NW];                           // survivors of tile w; -1: lists overflowed, -2: no such tile
    int next_task;
    int tile_active[NW];                      // is the ego agent of tile w active
    uint32_t tile_ntris[NW];                  // triangles of its environment's map as given (box primitive indices start there)
    Job tile_job[NW];                         // tile w, decoded by its warp
    Cam cam[NW];                              // its camera
};
static_assert(sizeof(FusedSmem) <= 44 * 1024 && sizeof(TileSmem) <= 44 * 1024,
              "shared memory must leave room for 5 CTAs per SM (228 KB, 1 KB reserved per CTA)");
// What the raster and store templates need of a warp's strip: rows are counted from the strip's first.
struct StripView {
    unsigned long long* key;
    const float* ray_x;
    const float* ray_y;
};
constexpr size_t RENDER_SMEM_BASE = sizeof(FusedSmem) > sizeof(TileSmem) ? sizeof(FusedSmem) : sizeof(TileSmem);

__device__ __forceinline__ void write_record(float4* r, const PrimEq& q, uint32_t key_lo, uint32_t box, uint32_t extra) {
    const uint32_t bx0 = box & 0xff, by0 = (box >> 8) & 0xff, bx1 = (box >> 16) & 0xff, by1 = box >> 24;
    r[0] = make_float4(q.nx[0], q.nx[1], q.nx[2], q.nx[3]);
    r[1] = make_float4(q.ny[0], q.ny[1], q.ny[2], q.ny[3]);
    r[2] = make_float4(q.nz[0], q.nz[1], q.nz[2], q.nz[3]);
    r[3] = make_float4(q.wx, q.wy, q.wz, __uint_as_float(key_lo));
    // the pixel box needs 6 bits per coordinate; the top-left bits and the flags ride along
    r[4].x = __uint_as_float(bx0 | (by0 << 6) | (bx1 << 12) | (by1 << 18) | (q.tl << 24) | extra);
}

__device__ __forceinline__ void read_record(const float4* r, PrimEq& q, uint32_t& key_lo) {
    const float4 r0 = r[0], r1 = r[1], r2 = r[2], r3 = r[3];
    q.nx[0] = r0.x; q.nx[1] = r0.y; q.nx[2] = r0.z; q.nx[3] = r0.w;
    q.ny[0] = r1.x; q.ny[1] = r1.y; q.ny[2] = r1.z; q.ny[3] = r1.w;
    q.nz[0] = r2.x; q.nz[1] = r2.y; q.nz[2] = r2.z; q.nz[3] = r2.w;
    q.wx = r3.x; q.wy = r3.y; q.wz = r3.z;
    key_lo = __float_as_uint(r3.w);
}

// Box test against planes held in registers (see box_visible).
__device__ __forceinline__ bool box_visible_reg(const float4 (&pl)[6], float px, float py, const Node& b) {
    const float ax = sub(b.lo[0], px), bx = sub(b.hi[0], px);
    const float ay = sub(b.lo[1], py), by = sub(b.hi[1], py);
    const float cx = 0.5f * (ax + bx), cy = 0.5f * (ay + by), cz = 0.5f * (b.lo[2] + b.hi[2]);
    const float hx = 0.5f * (bx - ax), hy = 0.5f * (by - ay), hz = 0.5f * (b.hi[2] - b.lo[2]);
    const float slack = 1e-3f + 4e-6f * (fabsf(cx) + fabsf(cy) + fabsf(cz) + hx + hy + hz);
    bool vis = true;
#pragma unroll
    for (int p = 0; p < 6; ++p) {
        const float dist = pl[p].x * cx + pl[p].y * cy + pl[p].z * cz + pl[p].w;
        const float reach = fabsf(pl[p].x) * hx + fabsf(pl[p].y) * hy + fabsf(pl[p].z) * hz;
        vis = vis && (dist + reach >= -slack);
    }
    return vis;
}

__device__ __forceinline__ Node load_node(const Node* p) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(p)), b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    Node nd;
    nd.lo[0] = a.x; nd.lo[1] = a.y; nd.lo[2] = a.z; nd.first = __float_as_uint(a.w);
    nd.hi[0] = b.x; nd.hi[1] = b.y; nd.hi[2] = b.z; nd.count = __float_as_uint(b.w);
    return nd;
}

__device__ __forceinline__ AgentGeom load_agent(const AgentGeom* p) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(p)), b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    AgentGeom g;
    g.x = a.x; g.y = a.y; g.c = a.z; g.s = a.w; g.hl = b.x; g.hw = b.y; g.h = b.z; g.active = __float_as_uint(b.w);
    return g;
}

__device__ __forceinline__ bool tiny_box(uint32_t box) {
    const int bx0 = box & 0xff, by0 = (box >> 8) & 0xff, bx1 = (box >> 16) & 0xff, by1 = box >> 24;
    return (bx1 - bx0 + 1) * (by1 - by0 + 1) <= TINY_MAX_PIXELS;
}

// Warp-wide append to the two-ended survivor list (see SURV_STRIDE).
__device__ __forceinline__ void append_survivor(uint2* __restrict__ surv, bool keep, uint32_t id, uint32_t box, int& n_big, int& n_tiny, int lane) {
    const bool tiny = keep && tiny_box(box), big = keep && !tiny;
    const unsigned mb = __ballot_sync(0xffffffffu, big), mt = __ballot_sync(0xffffffffu, tiny);
    const unsigned below = (1u << lane) - 1u;
    // (a slot is written only while front and back have not met; the caller checks the total)
    if (big) { const int slot = n_big + __popc(mb & below); if (slot + n_tiny < W_SURV) surv[slot] = make_uint2(id, box); }
    if (tiny) { const int slot = n_tiny + __popc(mt & below); if (slot + n_big + __popc(mb) < W_SURV) surv[W_SURV - 1 - slot] = make_uint2(id, box); }
    n_big += __popc(mb);
    n_tiny += __popc(mt);
}

// Front end of one tile by one warp: fills the survivor list.  Returns the survivor counts
// (front | back << 16), or -1 if a list overflowed (the tile then goes to the cooperative kernel).
//
// Map primitives come from the uniform grid: the footprint of the tile's frustum on the ground
// plane is the convex hull of the apex and the four far corners; for every grid row the footprint
// (widened by the map's margin) crosses, the small primitives of the cells it covers are one
// contiguous range of cell_prims.  The ranges of up to 32 rows are laid end to end and tested two
// candidates per lane at a time (camera space, pixel box).  The large primitives are found through
// their leaves (a lane per leaf box against the six frustum planes), the other agents' boxes as
// bounding spheres.  Loads that do not depend on one another are issued together.
template <class TL, bool CONS>
__device__ __forceinline__ int front_cull(FrontLists& f, uint2* __restrict__ surv, const RenderParams& P, const Job& job,
                                          const MapInfo& mi, int lane, TL& n) {
    const int stop = PIC_STOP(P);
    // CONS: conservative pixel boxes -- every pixel whose unit square a primitive touches (antialiased output)
    constexpr float BOX_MARGIN = CONS ? 0.50390625f : 0.00390625f;
    const TileCtx& t = job.t;
    const AgentGeom* env_agents = P.agents + (size_t)job.e * P.A;
    Node ln0;
    ln0.first = 0; ln0.count = 0;
    if (mi.large_begin + lane < mi.large_end) ln0 = load_node(P.large_leaves + mi.large_begin + lane);
    AgentGeom ag0, ag1;
    ag0.active = 0u; ag1.active = 0u;
    if (lane < P.A) ag0 = load_agent(env_agents + lane);
    if (lane + 32 < P.A) ag1 = load_agent(env_agents + lane + 32);
    if (lane < 7) {
        Cam c;
        load_camera(c, P.cams[job.view], P.cam[job.k], P.W, P.H);
        if (lane == 6) { f.cam = c; f.n_face = 0; }
        else tile_planes(f, lane, c, t);
        if (lane < 5) {
            // footprint corner `lane`: the apex, or a corner of the tile's frustum at depth far (a little beyond)
            const float F = lane ? t.far_z * 1.001f : 0.f;
            const float xc = ((float)((lane & 1) ? t.x0 + t.tw : t.x0) - c.cx) / c.focx * F;
            const float yc = ((float)((lane & 2) ? t.y0 + t.th : t.y0) - c.cy) / c.focy * F;
            f.pt[lane][0] = c.mwx + c.rx * xc + c.dx * yc + c.fx_ * F;
            f.pt[lane][1] = c.mwy + c.ry * xc + c.dy * yc + c.fy_ * F;
        }
    }
    __syncwarp();
    if (lane < 10) {
        // segment between two of the five corners (every pair: the hull's edges are among them, the others lie inside it)
        const int i = lane < 4 ? 0 : lane < 7 ? 1 : lane < 9 ? 2 : 3, j = lane < 4 ? lane + 1 : lane < 7 ? lane - 2 : lane < 9 ? lane - 4 : 4;
        const float px = f.pt[i][0], py = f.pt[i][1], dx = f.pt[j][0] - px, dy = f.pt[j][1] - py;
        f.seg[lane][0] = px; f.seg[lane][1] = py; f.seg[lane][2] = dx; f.seg[lane][3] = dy;
        f.seg[lane][4] = dy != 0.f ? 1.f / dy : 0.f; f.seg[lane][5] = 0.f;
    }
    __syncwarp();
    if (stop == 11) return 0;
    const Cam& c = f.cam;
    int n_big = 0, n_tiny = 0;
    // ---- the grid rows crossed by the widened footprint; the range of a row's cells in grid_prims
    const float margin = mi.margin, gx0 = sub(mi.gx0, c.px), gy0 = sub(mi.gy0, c.py);
    float ylo = f.pt[0][1], yhi = ylo;
#pragma unroll
    for (int k = 1; k < 5; ++k) { ylo = fminf(ylo, f.pt[k][1]); yhi = fmaxf(yhi, f.pt[k][1]); }
    const float fr0 = floorf((ylo - margin - gy0) * mi.inv_cell), fr1 = floorf((yhi + margin - gy0) * mi.inv_cell);
    const int row_lo = (int)fmaxf(fr0, 0.f), row_hi = (int)fminf(fr1, (float)mi.ny - 1.f);     // (empty if the footprint misses the grid)
    auto row_range = [&](int row, uint32_t& first, uint32_t& cnt) {
        first = 0u; cnt = 0u;
        if (row > row_hi) return;
        ++n.grp;
        const float blo = gy0 + (float)row * mi.cell - margin, bhi = blo + mi.cell + 2.f * margin;
        float xlo = 3e38f, xhi = -3e38f;
#pragma unroll 1
        for (int k = 0; k < 10; ++k) {
            const float px = f.seg[k][0], py = f.seg[k][1], dx = f.seg[k][2], dy = f.seg[k][3], idy = f.seg[k][4];
            const float ya = fminf(py, py + dy), yb = fmaxf(py, py + dy);
            if (yb >= blo && ya <= bhi) {
                const float ta = (blo - py) * idy, tb = (bhi - py) * idy;
                const float t0 = dy != 0.f ? fminf(fmaxf(fminf(ta, tb), 0.f), 1.f) : 0.f, t1 = dy != 0.f ? fminf(fmaxf(fmaxf(ta, tb), 0.f), 1.f) : 1.f;
                const float xa = px + t0 * dx, xb = px + t1 * dx;
                xlo = fminf(xlo, fminf(xa, xb)); xhi = fmaxf(xhi, fmaxf(xa, xb));
            }
        }
        if (xlo <= xhi) {
            const float fx0 = floorf((xlo - margin - gx0) * mi.inv_cell), fx1 = floorf((xhi + margin - gx0) * mi.inv_cell);
            if (fx1 >= 0.f && fx0 <= (float)mi.nx - 1.f) {
                const uint32_t ix0 = (uint32_t)fmaxf(fx0, 0.f), ix1 = (uint32_t)fminf(fx1, (float)mi.nx - 1.f);
                const uint32_t* cs = P.cell_start + mi.cell_begin + (uint32_t)row * mi.nx;
                first = __ldg(cs + ix0);
                cnt = __ldg(cs + ix1 + 1) - first;
            }
        }
    };
    // the first 32 rows' ranges are requested now; the boxes below are tested while the loads are under way
    uint32_t first0, cnt0;
    row_range(row_lo + lane, first0, cnt0);
    // ---- the large primitives' leaves: a lane per leaf box against the six frustum planes
    int n_ll = 0;
    {
        float4 pl[6];
#pragma unroll
        for (int p = 0; p < 6; ++p) pl[p] = *reinterpret_cast<const float4*>(f.plane[p]);
        for (uint32_t l0 = mi.large_begin; l0 < mi.large_end; l0 += 32) {
            const uint32_t l = l0 + lane;
            bool vis = false;
            Node ln;
            ln.first = 0; ln.count = 0;
            if (l < mi.large_end) { ln = (l0 == mi.large_begin) ? ln0 : load_node(P.large_leaves + l); vis = box_visible_reg(pl, c.px, c.py, ln); ++n.leaf; }
            const unsigned m = __ballot_sync(0xffffffffu, vis);
            if (vis) {
                const int slot = n_ll + __popc(m & ((1u << lane) - 1u));
                if (slot < W_LARGE) f.lleaf[slot] = (ln.first << 3) | ln.count;
            }
            n_ll += __popc(m);
        }
        if (n_ll > W_LARGE) return -1;
    }
    // ---- other agents' boxes, two per lane at a time
    for (int b0 = 0; b0 < P.A; b0 += 64) {
        if (b0 > 0) {
            ag0.active = 0u; ag1.active = 0u;
            if (b0 + lane < P.A) ag0 = load_agent(env_agents + b0 + lane);
            if (b0 + lane + 32 < P.A) ag1 = load_agent(env_agents + b0 + lane + 32);
        }
#pragma unroll 1
        for (int u = 0; u < 2; ++u) {
            const AgentGeom g = u ? ag1 : ag0;
            const int b = b0 + lane + 32 * u;
            uint32_t faces = 0u;
            if (b < P.A && b != job.a && g.active) faces = box_faces(f, c, t, g);
            if (faces) {
                int slot = atomicAdd(&f.n_face, __popc(faces));
                for (; faces; faces &= faces - 1, ++slot)
                    if (slot < W_FACE) f.face[slot] = ((uint32_t)b << 3) | (uint32_t)(__ffs(faces) - 1);
            }
        }
    }
    if (stop == 12) return 0;
    // ---- candidates of the grid rows, 32 rows per pass: camera space, pixel box; survivors are compacted
    for (int r0 = row_lo; r0 <= row_hi; r0 += 32) {
        uint32_t first = first0, cnt = cnt0;
        if (r0 != row_lo) row_range(r0 + lane, first, cnt);
        uint32_t incl = cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        const int total = (int)__shfl_sync(0xffffffffu, incl, 31);
        __syncwarp();
        f.row_first[lane] = first;
        f.row_off[lane] = incl - cnt;
        if (lane == 31) f.row_off[32] = incl;
        __syncwarp();
        for (int i0 = 0; i0 < total; i0 += 64) {         // two candidates per lane at a time
            float v[2][12];
            bool have[2];
            uint32_t id[2] = {0u, 0u};
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int i = i0 + 32 * u + lane;
                have[u] = i < total;
                if (have[u]) {
                    int r = 0;
#pragma unroll
                    for (int st = 16; st; st >>= 1)
                        if (f.row_off[r + st] <= (uint32_t)i) r += st;
                    id[u] = f.row_first[r] + ((uint32_t)i - f.row_off[r]);
                    uint32_t key_lo, flags;
                    load_prim(P.grid_prims + id[u], v[u], key_lo, flags);
                }
            }
#pragma unroll 1
            for (int u = 0; u < 2; ++u) {               // (one copy of the test for both candidates: less code to fetch)
                uint32_t box = 0;
                bool keep = false;
                const bool hv = u ? have[1] : have[0];
                if (hv) {
                    V3 V[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        V[q] = to_camera(c, u ? v[1][3 * q] : v[0][3 * q], u ? v[1][3 * q + 1] : v[0][3 * q + 1], u ? v[1][3 * q + 2] : v[0][3 * q + 2]);
                    ++n.tested;
                    keep = pixel_box(c, t, V, box, BOX_MARGIN);
                }
                append_survivor(surv, keep, u ? id[1] : id[0], box, n_big, n_tiny, lane);
            }
        }
    }
    // ---- the primitives of the visible large leaves
    __syncwarp();
    for (int i0 = 0; i0 < n_ll * LARGE_LEAF_PRIMS; i0 += 32) {
        const int i = i0 + lane;
        uint32_t box = 0, id = 0;
        bool keep = false;
        if (i < n_ll * LARGE_LEAF_PRIMS) {
            const uint32_t lf = f.lleaf[i / LARGE_LEAF_PRIMS];
            const uint32_t j = i % LARGE_LEAF_PRIMS;
            if (j < (lf & 7u)) {
                id = (lf >> 3) + j;
                float v[12];
                uint32_t key_lo, flags;
                load_prim(P.grid_prims + id, v, key_lo, flags);
                V3 V[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) V[q] = to_camera(c, v[3 * q], v[3 * q + 1], v[3 * q + 2]);
                ++n.tested;
                keep = pixel_box(c, t, V, box, BOX_MARGIN);
            }
        }
        append_survivor(surv, keep, id, box, n_big, n_tiny, lane);
    }
    __syncwarp();
    const int n_face = f.n_face;
    if (n_face > W_FACE) return -1;
    if (stop == 13) return 0;
    for (int i0 = 0; i0 < n_face; i0 += 32) {
        const int i = i0 + lane;
        uint32_t box = 0, it = 0;
        bool keep = false;
        if (i < n_face) {
            it = f.face[i];
            const AgentGeom g = load_agent(env_agents + (it >> 3));
            const uint32_t corners = face_corners((int)(it & 7u));
            V3 V[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) V[q] = box_corner(c, g, (corners >> (4 * q)) & 7u);
            ++n.tested;
            keep = pixel_box(c, t, V, box, BOX_MARGIN);
        }
        append_survivor(surv, keep, SURV_FACE | it, box, n_big, n_tiny, lane);
    }
    __syncwarp();
    if (stop == 14) return 0;
    return n_big + n_tiny > W_SURV ? -1 : (n_big | (n_tiny << 16));
}

// Survivor `id` in camera space with its plane normal.
__device__ __forceinline__ void fetch_survivor(const Cam& c, const RenderParams& P, uint32_t id, int e, uint32_t n_map_tris,
                                               V3 (&V)[4], V3& Pn, uint32_t& key_lo, uint32_t& flags) {
    if (!(id & SURV_FACE)) {
        float v[12], vis_cos;
        load_prim(P.grid_prims + id, v, key_lo, flags, vis_cos);
#pragma unroll
        for (int q = 0; q < 4; ++q) V[q] = to_camera(c, v[3 * q], v[3 * q + 1], v[3 * q + 2]);
        Pn = limit_angular_range(V, plane_normal_world(c, v, flags & 1u), vis_cos);
    } else {
        const int b = (int)((id & ~SURV_FACE) >> 3), f = (int)(id & 7u);
        const AgentGeom g = P.agents[(size_t)e * P.A + b];
        const uint32_t corners = face_corners(f);
#pragma unroll
        for (int q = 0; q < 4; ++q) V[q] = box_corner(c, g, (corners >> (4 * q)) & 7u);
        key_lo = ((0xFFFFFFu - (n_map_tris + 12u * (uint32_t)b + 2u * (uint32_t)f)) << 8) | agent_box_class(g);
        flags = face_flags(corners);
        Pn = plane_normal(V, true);
    }
}

// A covered pixel's depth lies between the vertices' depths; with a margin far above the rounding
// of the 1/z plane, vertices well inside [near, far] make the per-pixel range test redundant.
__device__ __forceinline__ bool record_in_range(const V3 (&V)[4], const RenderParams& P) {
    const float zlo = fminf(fminf(V[0].z, V[1].z), fminf(V[2].z, V[3].z)), zhi = fmaxf(fmaxf(V[0].z, V[1].z), fmaxf(V[2].z, V[3].z));
    return zlo >= P.near_z * 1.001f && zhi <= P.far_z * 0.999f;
}

// Set-up of a tile's survivors (the cull kernel's list) by its warp: survivor i becomes record i of `rec`.
template <class TL>
__device__ __forceinline__ void front_setup(const Cam& c, const uint2* __restrict__ surv, float4* rec, const RenderParams& P,
                                            const Job& job, const MapInfo& mi, int ns, int n_big, int lane, TL& n) {
    for (int i = lane; i < ns; i += 32) {
        const uint2 sv = __ldcg(surv + (i < n_big ? i : W_SURV - 1 - (i - n_big)));
        V3 V[4], Pn;
        uint32_t key_lo, flags;
        fetch_survivor(c, P, sv.x, job.e, mi.n_tris, V, Pn, key_lo, flags);
        PrimEq q;
        float4* r = rec + i * (REC / 4);
        if (!prim_equations(V, flags & 1u, flags, Pn, q)) { r[4].x = __uint_as_float(REC_DEAD); continue; }
        ++n.setup;
        const uint32_t box = sv.y;
        const int bx0 = box & 0xff, by0 = (box >> 8) & 0xff, bx1 = (box >> 16) & 0xff, by1 = box >> 24;
        const bool tiny = (bx1 - bx0 + 1) * (by1 - by0 + 1) <= TINY_MAX_PIXELS;
        if (tiny) ++n.tiny; else ++n.recs;
        write_record(r, q, key_lo, box, (tiny ? REC_TINY : 0u) | (record_in_range(V, P) ? REC_INRANGE : 0u));
    }
}

// Back end of one strip (rows ys .. ys + STRIP - 1 of the tile) by one warp; the strip's keys are
// all "no fragment" on entry and on exit.
template <bool FULL, class TL>
__device__ __forceinline__ void back_strip(StripView& s, const RenderParams& P, const Job& job, bool ego_active, int ys,
                                           const float4* rec, int n_rec, bool classify, int stop, int lane, uint32_t n_map_tris, TL& n) {
    const TileCtx& t = job.t;
    const int rows = FULL ? STRIP : min(STRIP, t.th - ys);
    uint32_t touched = 0u;                       // 8x8 blocks of the strip: bit (row >> 3) * 8 + (column >> 3)
    // Records are looked at 32 at a time, a lane each: which reach the strip?  Those of a few
    // pixels are rasterized by their lane (atomic max); the warp then walks the other hits
    // together, a lane per pixel pair.
    for (int base = 0; base < n_rec; base += 32) {
        uint32_t bw_lane = 0u;
        bool hit = false;
        if (base + lane < n_rec) {
            const float4* r = rec + (base + lane) * (REC / 4);
            bw_lane = __float_as_uint(r[4].x);
            const int by0 = (bw_lane >> 6) & 63, by1 = (bw_lane >> 18) & 63;
            hit = !(bw_lane & REC_DEAD) && by1 >= ys && by0 < ys + STRIP;
            if (hit && (bw_lane & REC_TINY) && stop == 7) hit = false;
            if (hit && (bw_lane & REC_TINY)) {
                hit = false;
                const int bx0 = bw_lane & 63, bx1 = (bw_lane >> 12) & 63;
                const int y0 = max(by0, ys) - ys, y1 = min(by1, ys + STRIP - 1) - ys;
                PrimEq q;
                uint32_t key_lo;
                read_record(r, q, key_lo);
                q.tl = (bw_lane >> 24) & 15u;
                // at most TINY_MAX_PIXELS pixels: one column (w == 1), two columns, or one row
                const int w = bx1 - bx0 + 1, npx = w * (y1 - y0 + 1);
                bool any = false;
#pragma unroll
                for (int px = 0; px < TINY_MAX_PIXELS; ++px) {
                    if (px < npx) {
                        const int x = bx0 + (w == 1 ? 0 : w == 2 ? (px & 1) : px), y = y0 + (w == 1 ? px : w == 2 ? (px >> 1) : 0);
                        const uint32_t wb = fragment(q, s.ray_x[x], s.ray_y[y], t.w_near, t.w_far);
                        if (wb) { put_fragment(s, x, y, wb, key_lo); any = true; }
                    }
                }
                if (any) touched |= (uint32_t)block_mask(bx0, y0, bx1, y1);
            }
        }
        __syncwarp();
        unsigned hits = __ballot_sync(0xffffffffu, hit);
        if (!(stop == 0 || stop > 5)) hits = 0u;
        for (; hits; hits &= hits - 1) {
            const int src = __ffs(hits) - 1;
            const uint32_t bw = __shfl_sync(0xffffffffu, bw_lane, src);
            const float4* r = &rec[(base + src) * (REC / 4)];
            const int by0 = (bw >> 6) & 63, by1 = (bw >> 18) & 63;
            const int bx0 = bw & 63, bx1 = (bw >> 12) & 63;
            const int ly0 = max(by0, ys) - ys, ly1 = min(by1, ys + STRIP - 1) - ys;
            PrimEq q;
            uint32_t key_lo;
            read_record(r, q, key_lo);
            q.tl = (bw >> 24) & 15u;
            float thr[4];
            edge_thresholds(q.tl, thr);
            if (classify && (bx1 - bx0 + 1) * (ly1 - ly0 + 1) >= CLASSIFY_MIN_STRIP) {
                // lanes 0..15 classify the strip's 16 x 4 pixel cells: reject / partly covered / inside
                ++n.classified;
                const int xa = (lane & 3) * 16, xb = xa + 15, ya = ((lane >> 2) & 3) * 4, yb = ya + 3;
                bool reject = lane >= 16 || xb < bx0 || xa > bx1 || yb < ly0 || ya > ly1;
                uint32_t need = 0u;
                if (!reject) {
                    const float rxa = s.ray_x[xa], rxb = s.ray_x[xb], rya = s.ray_y[ya], ryb = s.ray_y[yb];   // rxa < rxb, rya < ryb
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        // fma is monotone in each argument, so the cell's extreme values are at its corners
                        const float ta = fm(q.ny[e], rya, q.nz[e]), tb = fm(q.ny[e], ryb, q.nz[e]);
                        const float emax = fm(q.nx[e], q.nx[e] >= 0.f ? rxb : rxa, fmaxf(ta, tb));
                        const float emin = fm(q.nx[e], q.nx[e] >= 0.f ? rxa : rxb, fminf(ta, tb));
                        reject = reject || (emax < 0.f);
                        if (!(emin > 0.f)) need |= 1u << e;
                    }
                    const float wa = fm(q.wy, rya, q.wz), wb = fm(q.wy, ryb, q.wz);
                    const float wmax = fm(q.wx, q.wx >= 0.f ? rxb : rxa, fmaxf(wa, wb));
                    const float wmin = fm(q.wx, q.wx >= 0.f ? rxa : rxb, fminf(wa, wb));
                    reject = reject || (wmax < t.w_far) || (wmin > t.w_near);
                    // the depth range test rides on the edge tests: if it is still needed, so is one edge
                    if (need == 0u && !((wmin >= t.w_far) && (wmax <= t.w_near))) need = 1u;
                }
                for (unsigned m = __ballot_sync(0xffffffffu, !reject); m; m &= m - 1) {
                    const int cell = __ffs(m) - 1;
                    const int xx = (cell & 3) * 16, yy = (cell >> 2) * 4;
                    const uint32_t need_c = __shfl_sync(0xffffffffu, need, cell);
                    ++n.cells;
                    if (raster_cell(s, t, q, thr, key_lo, xx, yy, need_c, lane)) touched |= 3u << ((yy >> 3) * 8 + (xx >> 3));
                }
            } else {
                for (int yy = ly0 & ~3; yy <= ly1; yy += 4)
                    for (int xx = bx0 & ~15; xx <= bx1; xx += 16) {
                        ++n.cells;
                        if (raster_cell(s, t, q, thr, key_lo, xx, yy, 0xFu, lane)) touched |= 3u << ((yy >> 3) * 8 + (xx >> 3));
                    }
            }
        }
        __syncwarp();
    }
    touched = __reduce_or_sync(0xffffffffu, touched);
    if (stop == 5) touched = 0xffffu;
    // ---- store; a ragged strip may hold keys past the image edge, which the store never visits:
    // it clears the whole strip instead of the keys it read
    TileCtx ts = t;
    ts.y0 = t.y0 + ys; ts.th = rows;
    const bool ragged = !FULL && (t.tw < TILE || rows < STRIP);
    if (stop != 8) store_tile<FULL>(s, ts, P, job.view, job.k, ego_active, (unsigned long long)touched, !ragged, lane, 32, n_map_tris);
    __syncwarp();
    if (ragged) {
#pragma unroll
        for (int i = 0; i < STRIP_KEYS / 2 / 32; ++i)
            reinterpret_cast<ulonglong2*>(s.key)[i * 32 + lane] = make_ulonglong2(0ull, 0ull);
        __syncwarp();
    }
}

// Cull kernel: a warp per tile walks the hierarchy and the other agents' boxes, tests the candidates
// and leaves the tile's survivors (id, pixel box) in device memory: a 16-byte head (count, or -1 if a
// list overflowed; with counters, the tile's group / leaf / candidate tests), then the list.  No
// CTA-wide synchronisation.  The lists are small (about 250 bytes per view on the benchmark
// workload) and are read back by the render kernel that follows on the stream.
struct __align__(16) CullSmem {
    FrontLists lists[NW];
};

#ifndef PIC_CULL_CTAS
#define PIC_CULL_CTAS 6
#endif
#ifndef PIC_CULL_ROUNDS
#define PIC_CULL_ROUNDS 1
#endif
constexpr int CULL_ROUNDS = PIC_CULL_ROUNDS;   // rounds of NW tiles per CTA of the cull kernel
#ifndef PIC_RENDER_CTAS
#define PIC_RENDER_CTAS 5
#endif
template <class TL, bool CONS>
__global__ void __launch_bounds__(NTHREADS, PIC_CULL_CTAS) cull_kernel(const __grid_constant__ RenderParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    CullSmem& s = *reinterpret_cast<CullSmem*>(smem_raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stop = PIC_STOP(P);
    // a CTA takes CULL_ROUNDS x NW consecutive tiles, NW at a time: consecutive tiles belong to the
    // same or to neighbouring agents, so the map data a round pulls in serves the next from L1
#pragma unroll 1
    for (int round = 0; round < CULL_ROUNDS; ++round) {
        const unsigned id = (blockIdx.x * (unsigned)CULL_ROUNDS + round) * (unsigned)NW + warp;
        if (id >= P.n_jobs) return;
        TL n = {};
        const Job job = decode_job(P, id);
        const MapInfo mi = P.env_maps[job.e];
        const bool ego_active = P.agents[(size_t)job.e * P.A + job.a].active != 0;
        uint2* blk = P.surv + (size_t)id * SURV_STRIDE;
        int ns = 0;
        if (P.debug_flags & 4) ns = -1;             // test aid: every tile through cooperative_job
        else if (ego_active && stop != 1 && !(stop >= 8 && stop <= 10)) ns = front_cull<TL, CONS>(s.lists[warp], blk + 2, P, job, mi, lane, n);
        // (the work counts are summed over the warp's lanes; without counters they are constants)
        const uint32_t c_grp = __reduce_add_sync(0xffffffffu, (uint32_t)tally_value(n.grp)), c_leaf = __reduce_add_sync(0xffffffffu, (uint32_t)tally_value(n.leaf)),
                       c_tested = __reduce_add_sync(0xffffffffu, (uint32_t)tally_value(n.tested));
        if (lane == 0) *reinterpret_cast<uint4*>(blk) = make_uint4((uint32_t)ns, c_grp, c_leaf, c_tested);
        __syncwarp();
    }
}

// Render kernel.  FULL: every tile is 64 x 64, rows allow 128-bit stores, no float32 depth image (the
// launcher checks) -- the instantiation the workloads run, without the code for ragged tiles.
template <class TL, bool FULL>
__global__ void __launch_bounds__(NTHREADS, 5) render_kernel(const __grid_constant__ RenderParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    FusedSmem& s = *reinterpret_cast<FusedSmem*>(smem_raw);
    if (PIC_STOP(P) == 15) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned first = blockIdx.x * (unsigned)NW, n_jobs = P.n_jobs;
    TL n = {};
    const bool classify = !(P.debug_flags & 1);
    const int stop = PIC_STOP(P);
    // test aids: a pool of 2 records sends nearly every tile to cooperative_job, one of 40 mixes both paths
    const int pool_cap = FULL ? POOL : (P.debug_flags & 2) ? 2 : (P.debug_flags & 8) ? 40 : POOL;   // (FULL is launched without these flags)
    if (threadIdx.x == 0) s.next_task = 0;

    // ---- the cull kernel's survivors of tile first + w
    const bool valid = first + warp < n_jobs;
    Job job;
    MapInfo mi;
    const uint2* blk = P.surv + (size_t)(first + warp) * SURV_STRIDE;
    int ns = -2, n_big = 0;
    if (valid) {
        const uint4 head = __ldcg(reinterpret_cast<const uint4*>(blk));
        job = decode_job(P, first + warp);
        mi = P.env_maps[job.e];
        const bool ego_active = P.agents[(size_t)job.e * P.A + job.a].active != 0;
        if (lane == 0) {
            s.tile_job[warp] = job; s.tile_active[warp] = ego_active; s.tile_ntris[warp] = mi.n_tris;
            load_camera(s.cam[warp], P.cams[job.view], P.cam[job.k], P.W, P.H);
        }
        n_big = (int)(head.x & 0xffffu);
        ns = head.x == SURV_OVERFLOW ? -1 : n_big + (int)(head.x >> 16);
        if (lane == 0) { n.grp = (int)head.y; n.leaf = (int)head.z; n.tested = (int)head.w; }
    }
    if (lane == 0) s.n_surv[warp] = ns;
    __syncthreads();
    // every thread lays the record pool out alike: tiles in order, a tile that does not fit is left
    // out.  One byte per tile: first record, and count (0xff: to cooperative_job, 0xfe: no such tile)
    uint32_t bases = 0u, cnts = 0u;
    {
        int off = 0;
#pragma unroll
        for (int j = 0; j < NW; ++j) {
            const int c = s.n_surv[j];
            bases |= (uint32_t)off << (8 * j);
            if (c >= 0 && off + c <= pool_cap) { cnts |= (uint32_t)c << (8 * j); off += c; }
            else cnts |= ((c == -2) ? 0xfeu : 0xffu) << (8 * j);
        }
    }
    {
        const int my_base = (int)((bases >> (8 * warp)) & 0xffu), my_cnt = (int)((cnts >> (8 * warp)) & 0xffu);
        if (my_cnt == 0xff) { n.grp = 0; n.leaf = 0; n.tested = 0; }       // counted again by cooperative_job
        else if (my_cnt != 0xfe && my_cnt > 0 && stop != 14) front_setup(s.cam[warp], blk + 2, s.pool + my_base * (REC / 4), P, job, mi, my_cnt, n_big, lane, n);
    }
    __syncthreads();
    // ---- back end: the NW tiles' strips are tasks that the warps draw from a counter; a warp's
    // lists are dead, their memory becomes its strip of keys
    if (stop != 9) {
#pragma unroll
        for (int i = 0; i < STRIP_KEYS / 2 / 32; ++i)
            reinterpret_cast<ulonglong2*>(s.key[warp])[i * 32 + lane] = make_ulonglong2(0ull, 0ull);
    }
    __syncwarp();
    if (stop == 10) return;
    StripView sv;
    sv.key = s.key[warp]; sv.ray_x = s.ray_x[warp]; sv.ray_y = s.ray_y[warp];
    constexpr int STRIPS = TILE / STRIP;
#pragma unroll 1
    for (;;) {
        int task = 0;
        if (lane == 0) task = atomicAdd(&s.next_task, 1);
        task = __shfl_sync(0xffffffffu, task, 0);
        if (task >= NW * STRIPS) break;
        const int j = task / STRIPS, ys = (task % STRIPS) * STRIP;
        const int cj = (int)((cnts >> (8 * j)) & 0xffu);
        if (cj >= 0xfe) continue;
        const Job jb = s.tile_job[j];
        if (!FULL && ys >= jb.t.th) continue;
        const bool ego_active = s.tile_active[j] != 0;
        if (FULL || (jb.t.tw == TILE && ys + STRIP <= jb.t.th)) {     // ray tables of the strip
            const float* rx = P.rig.ray_x + (size_t)jb.k * P.W + jb.t.x0;
            s.ray_x[warp][lane] = __ldg(rx + lane);
            s.ray_x[warp][lane + 32] = __ldg(rx + lane + 32);
            if (lane < STRIP) s.ray_y[warp][lane] = __ldg(P.rig.ray_y + (size_t)jb.k * P.H + jb.t.y0 + ys + lane);
        } else {                                            // ragged: columns / rows past the image edge continue the formula
            const CamConst& ck = P.cam[jb.k];
#pragma unroll
            for (int i = lane; i < TILE; i += 32)
                s.ray_x[warp][i] = (jb.t.x0 + i < P.W) ? __ldg(P.rig.ray_x + (size_t)jb.k * P.W + jb.t.x0 + i)
                                                      : __fdiv_rn(sub(add((float)(jb.t.x0 + i), 0.5f), 0.5f * (float)P.W), ck.fx);
            if (lane < STRIP) {
                const int y = jb.t.y0 + ys + lane;
                s.ray_y[warp][lane] = (y < P.H) ? __ldg(P.rig.ray_y + (size_t)jb.k * P.H + y)
                                                : __fdiv_rn(sub(add((float)y, 0.5f), 0.5f * (float)P.H), ck.fy);
            }
        }
        __syncwarp();
        back_strip<FULL>(sv, P, jb, ego_active, ys, s.pool + ((bases >> (8 * j)) & 0xffu) * (REC / 4), cj, classify, stop, lane, s.tile_ntris[j], n);
        if (lane == 0 && ys == 0) ++n.jobs;
    }
    // ---- the rest: tiles that did not fit are left to the cooperative kernel
    if (threadIdx.x < NW && ((cnts >> (8 * threadIdx.x)) & 0xffu) == 0xffu)
        P.overflow[1u + atomicAdd(&P.overflow[0], 1u)] = first + threadIdx.x;
    flush_counters(P, n);
}

// ---------------------------------------------------------------------------------------------
// Render kernel for images made of full 64 x 64 tiles whose rows allow vector stores (every
// benchmark workload).  Like render_kernel, with less bookkeeping: ray tables of the four tiles are
// loaded once, per-tile constants are a 16-byte record, the background rows a lane stores are
// fetched before the strip is rasterized.  The record pool is handed out in rounds: tiles that do
// not fit beside their fellows are set up and rasterized in a further round of the same CTA (their
// survivors are already in device memory), so only a tile whose own survivors exceed the pool, or
// whose cull lists overflowed, is left to the cooperative kernel.
// ---------------------------------------------------------------------------------------------
#ifndef PIC_FSTRIP
#define PIC_FSTRIP 16
#endif
#ifndef PIC_FPOOL
#define PIC_FPOOL 144
#endif
constexpr int FPOOL = PIC_FPOOL;     // records shared by the four tiles of a CTA
constexpr int FSTRIP = PIC_FSTRIP;   // pixel rows of a strip: 16 or 8
constexpr int FSTRIP_KEYS = TILE * FSTRIP;
constexpr int FSTRIPS = TILE / FSTRIP;
static_assert(FSTRIP == 16 || FSTRIP == 8, "strips of 16 or 8 rows");

// The record pool of the full-tile kernel, one array per 16-byte part of a record: 17 words per
// record instead of the 20 of an array of padded records, so more records fit beside the keys.
struct __align__(16) RecordPool {
    float4 nx[FPOOL], ny[FPOOL], nz[FPOOL];   // edge functions E_i = nx[i] rx + ny[i] ry + nz[i]
    float4 w[FPOOL];                          // 1/z plane wx, wy, wz; key low word
    uint32_t box[FPOOL];                      // pixel box (6 bits per coordinate), top-left bits, flags
};

__device__ __forceinline__ void write_record(RecordPool& pool, int slot, const PrimEq& q, uint32_t key_lo, uint32_t box, uint32_t extra) {
    const uint32_t bx0 = box & 0xff, by0 = (box >> 8) & 0xff, bx1 = (box >> 16) & 0xff, by1 = box >> 24;
    pool.nx[slot] = make_float4(q.nx[0], q.nx[1], q.nx[2], q.nx[3]);
    pool.ny[slot] = make_float4(q.ny[0], q.ny[1], q.ny[2], q.ny[3]);
    pool.nz[slot] = make_float4(q.nz[0], q.nz[1], q.nz[2], q.nz[3]);
    pool.w[slot] = make_float4(q.wx, q.wy, q.wz, __uint_as_float(key_lo));
    pool.box[slot] = bx0 | (by0 << 6) | (bx1 << 12) | (by1 << 18) | (q.tl << 24) | extra;
}

__device__ __forceinline__ void read_record(const RecordPool& pool, int slot, PrimEq& q, uint32_t& key_lo) {
    const float4 r0 = pool.nx[slot], r1 = pool.ny[slot], r2 = pool.nz[slot], r3 = pool.w[slot];
    q.nx[0] = r0.x; q.nx[1] = r0.y; q.nx[2] = r0.z; q.nx[3] = r0.w;
    q.ny[0] = r1.x; q.ny[1] = r1.y; q.ny[2] = r1.z; q.ny[3] = r1.w;
    q.nz[0] = r2.x; q.nz[1] = r2.y; q.nz[2] = r2.z; q.nz[3] = r2.w;
    q.wx = r3.x; q.wy = r3.y; q.wz = r3.z;
    key_lo = __float_as_uint(r3.w);
}

struct __align__(16) TileRef {
    size_t pixel0;       // offset of the tile's first pixel in the output images
    int bg_row0;         // first row of the tile in the per-camera background tables
    int active;          // is the ego agent active
};

struct __align__(16) FullSmem {
    unsigned long long key[NW][FSTRIP_KEYS];  // warp w's strip of keys
    RecordPool pool;
    float ray_x[NW][TILE], ray_y[NW][TILE];   // ray tables of tile w
    Cam cam[NW];
    TileRef tile[NW];
    int n_surv[NW];
    int next_task;
};
static_assert(sizeof(FullSmem) <= 44 * 1024, "shared memory must leave room for 5 CTAs per SM");

// The 16 x 4 cell of strip_cell's comment, for the full-tile kernel: `kbase` and `lsw` are the
// lane's share of the key address (row lane >> 3, chunk lane & 7, swizzle), `range` says whether
// the depth range still has to be tested (warp-uniform), keys are written with one predicated
// 64-bit store per pixel; the caller marks the touched blocks.
__device__ __forceinline__ void strip_cell(unsigned long long* key, const float* ray_x, const float* ray_y, const PrimEq& q,
                                           const float (&thr)[4], uint32_t key_lo, float w_near, float w_far, int xx, int yy,
                                           uint32_t need, bool range, int kbase, int lsw, int lane) {
    const float2 rx = *reinterpret_cast<const float2*>(ray_x + xx + (lane & 7) * 2);
    const float ry = ray_y[yy + (lane >> 3)];
    const float wt = fm(q.wy, ry, q.wz);
    const float w0 = fm(q.wx, rx.x, wt), w1 = fm(q.wx, rx.y, wt);
    bool in0 = true, in1 = true;
    if (need) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if ((need >> e) & 1u) {          // warp-uniform: edges known to be positive on the whole cell are skipped
                const float te = fm(q.ny[e], ry, q.nz[e]);
                const float e0 = fm(q.nx[e], rx.x, te), e1 = fm(q.nx[e], rx.y, te);
                in0 = in0 && (e0 > thr[e]);
                in1 = in1 && (e1 > thr[e]);
            }
        }
        if (range) {
            in0 = in0 && (w0 >= w_far) && (w0 <= w_near);
            in1 = in1 && (w1 >= w_far) && (w1 <= w_near);
        }
    }
    const int cb = xx >> 4;
    unsigned long long* kp = key + (kbase + (yy << 6) + (cb << 4) + ((lsw ^ cb) << 1));
    const ulonglong2 kk = *reinterpret_cast<const ulonglong2*>(kp);
    const unsigned long long k0 = make_key(__float_as_uint(w0), key_lo), k1 = make_key(__float_as_uint(w1), key_lo);
    if (in0 && k0 > kk.x) kp[0] = k0;
    if (in1 && k1 > kk.y) kp[1] = k1;
}

// Strip -> class / depth images, 16 pixels per lane and pass (see store_tile); resets the keys it reads.
__device__ __forceinline__ void store_strip_full(unsigned long long* key, uint8_t* oc, uint16_t* od, int W, uint32_t touched,
                                                 const uint32_t (&bgc)[2], const float (&bgz)[2], int lane) {
#pragma unroll
    for (int it = 0; it < FSTRIP / 8; ++it) {
        const int y = it * 8 + (lane >> 2), xs = (lane & 3) * 16;
        const size_t o = (size_t)y * W + xs;
        uint32_t cw[4], dw[8];
        if (((touched >> (it * 8 + (xs >> 3))) & 3u) == 0u) {       // both 8 x 8 blocks of the segment are background
            const uint32_t c4 = bgc[it] * 0x01010101u;
            const __half2 h = __floats2half2_rn(bgz[it], bgz[it]);
            const uint32_t d2 = *reinterpret_cast<const uint32_t*>(&h);
#pragma unroll
            for (int j = 0; j < 4; ++j) cw[j] = c4;
#pragma unroll
            for (int j = 0; j < 8; ++j) dw[j] = d2;
        } else {
#pragma unroll
            for (int j = 0; j < 16; j += 2) {
                ulonglong2* kp = reinterpret_cast<ulonglong2*>(&key[key_index(xs + j, y)]);
                const ulonglong2 kk = *kp;
                *kp = make_ulonglong2(0ull, 0ull);
                const float z0 = kk.x ? fast_rcp(__uint_as_float((uint32_t)(kk.x >> 32))) : bgz[it];
                const float z1 = kk.y ? fast_rcp(__uint_as_float((uint32_t)(kk.y >> 32))) : bgz[it];
                const uint32_t c0 = kk.x ? (uint32_t)(kk.x & 0xff) : bgc[it], c1 = kk.y ? (uint32_t)(kk.y & 0xff) : bgc[it];
                const __half2 h = __floats2half2_rn(z0, z1);
                dw[j >> 1] = *reinterpret_cast<const uint32_t*>(&h);
                if ((j & 3) == 0) cw[j >> 2] = c0 | (c1 << 8); else cw[j >> 2] |= (c0 << 16) | (c1 << 24);
            }
        }
#ifdef PIC_PROFILE
        if (touched & 0x80000000u) continue;       // profiling: no global stores
#endif
        *reinterpret_cast<uint4*>(oc + o) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
        store_256(od + o, dw);
    }
}

// One strip (rows ys .. of the tile) by one warp: the tile's fragments that fall into it, then
// the records that reach it, cell by cell.  Returns the touched 8 x 8 blocks.
__device__ __forceinline__ uint32_t raster_strip_full(StripView& s, const RecordPool& pool, int first, int n_rec, int ys, float w_near,
                                                      float w_far, int stop, int lane) {
    uint32_t touched = 0u;                       // bit (row >> 3) * 8 + (column >> 3)
    const int kbase = (lane >> 3) << 6, lsw = (lane & 7) ^ (((lane >> 3) & 1) << 2);   // see strip_cell
    for (int base = 0; base < n_rec; base += 32) {
        uint32_t bw_lane = 0u;
        bool hit = false;
        if (base + lane < n_rec) {
            const int slot = first + base + lane;
            bw_lane = pool.box[slot];
            const int by0 = (bw_lane >> 6) & 63, by1 = (bw_lane >> 18) & 63;
            hit = !(bw_lane & REC_DEAD) && by1 >= ys && by0 < ys + FSTRIP;
            if (hit && (bw_lane & REC_TINY)) {           // a few pixels: rasterized by this lane (atomic max)
                hit = false;
                const int bx0 = bw_lane & 63, bx1 = (bw_lane >> 12) & 63;
                const int y0 = max(by0, ys) - ys, y1 = min(by1, ys + FSTRIP - 1) - ys;
                PrimEq q;
                uint32_t key_lo;
                read_record(pool, slot, q, key_lo);
                q.tl = (bw_lane >> 24) & 15u;
                // at most TINY_MAX_PIXELS pixels: one column (w == 1), two columns, or one row
                const int w = bx1 - bx0 + 1, npx = (stop == 7) ? 0 : w * (y1 - y0 + 1);
                bool any = false;
#pragma unroll
                for (int px = 0; px < TINY_MAX_PIXELS; ++px) {
                    if (px < npx) {
                        const int x = bx0 + (w == 1 ? 0 : w == 2 ? (px & 1) : px), y = y0 + (w == 1 ? px : w == 2 ? (px >> 1) : 0);
                        const uint32_t wb = fragment(q, s.ray_x[x], s.ray_y[y], w_near, w_far);
                        if (wb) { put_fragment(s, x, y, wb, key_lo); any = true; }
                    }
                }
                if (any) touched |= (uint32_t)block_mask(bx0, y0, bx1, y1);
            }
        }
        __syncwarp();
        unsigned hits = __ballot_sync(0xffffffffu, hit);
        if (!(stop == 0 || stop == 2 || stop == 3 || stop > 5)) hits = 0u;
        for (; hits; hits &= hits - 1) {
            const int src = __ffs(hits) - 1;
            const uint32_t bw = __shfl_sync(0xffffffffu, bw_lane, src);
            const int by0 = (bw >> 6) & 63, by1 = (bw >> 18) & 63;
            const int bx0 = bw & 63, bx1 = (bw >> 12) & 63;
            const int ly0 = max(by0, ys) - ys, ly1 = min(by1, ys + FSTRIP - 1) - ys;
            PrimEq q;
            uint32_t key_lo;
            read_record(pool, first + base + src, q, key_lo);
            q.tl = (bw >> 24) & 15u;
            float thr[4];
            edge_thresholds(q.tl, thr);
            const bool range = !(bw & REC_INRANGE);
            if (stop != 3 && (bx1 - bx0 + 1) * (ly1 - ly0 + 1) >= CLASSIFY_MIN_STRIP * FSTRIP / 16) {
                // a lane per 16 x 4 pixel cell of the strip classifies it: reject / partly covered / inside
                const int xa = (lane & 3) * 16, xb = xa + 15, ya = ((lane >> 2) & 3) * 4, yb = ya + 3;
                bool reject = lane >= FSTRIP || xb < bx0 || xa > bx1 || yb < ly0 || ya > ly1;
                uint32_t need = 0u;
                if (!reject) {
                    const float rxa = s.ray_x[xa], rxb = s.ray_x[xb], rya = s.ray_y[ya], ryb = s.ray_y[yb];   // rxa < rxb, rya < ryb
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        // fma is monotone in each argument, so the cell's extreme values are at its corners
                        const float ta = fm(q.ny[e], rya, q.nz[e]), tb = fm(q.ny[e], ryb, q.nz[e]);
                        const float emax = fm(q.nx[e], q.nx[e] >= 0.f ? rxb : rxa, fmaxf(ta, tb));
                        const float emin = fm(q.nx[e], q.nx[e] >= 0.f ? rxa : rxb, fminf(ta, tb));
                        reject = reject || (emax < 0.f);
                        if (!(emin > 0.f)) need |= 1u << e;
                    }
                    const float wa = fm(q.wy, rya, q.wz), wb = fm(q.wy, ryb, q.wz);
                    const float wmax = fm(q.wx, q.wx >= 0.f ? rxb : rxa, fmaxf(wa, wb));
                    const float wmin = fm(q.wx, q.wx >= 0.f ? rxa : rxb, fminf(wa, wb));
                    reject = reject || (wmax < w_far) || (wmin > w_near);
                    // the depth range test rides on the edge tests: if it is still needed, so is one edge
                    if (need == 0u && !((wmin >= w_far) && (wmax <= w_near))) need = 1u;
                }
                for (unsigned m = __ballot_sync(0xffffffffu, !reject); m; m &= m - 1) {
                    const int cell = __ffs(m) - 1;
                    const int xx = (cell & 3) * 16, yy = (cell >> 2) * 4;
                    const uint32_t need_c = __shfl_sync(0xffffffffu, need, cell);
                    if (stop != 2 && stop != 3) strip_cell(s.key, s.ray_x, s.ray_y, q, thr, key_lo, w_near, w_far, xx, yy, need_c, true, kbase, lsw, lane);
                    touched |= 3u << ((yy >> 3) * 8 + (xx >> 3));
                }
            } else {
                for (int yy = ly0 & ~3; yy <= ly1; yy += 4)
                    for (int xx = bx0 & ~15; xx <= bx1; xx += 16)
                        if (stop != 2 && stop != 3) strip_cell(s.key, s.ray_x, s.ray_y, q, thr, key_lo, w_near, w_far, xx, yy, 0xFu, range, kbase, lsw, lane);
                touched |= (uint32_t)block_mask(bx0, ly0, bx1, ly1);
            }
        }
        __syncwarp();
    }
    return __reduce_or_sync(0xffffffffu, touched);
}

__global__ void __launch_bounds__(NTHREADS, PIC_RENDER_CTAS) render_full_kernel(const __grid_constant__ RenderParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    FullSmem& s = *reinterpret_cast<FullSmem*>(smem_raw);
    const int stop = PIC_STOP(P);
    if (stop == 15) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned id = blockIdx.x * (unsigned)NW + warp;
    const bool valid = id < P.n_jobs;
    // ---- the cull kernel's survivors of tile first + w, and everything that does not depend on them
    const uint2* blk = P.surv + (size_t)id * SURV_STRIDE;
    int ns = -2, n_big = 0;
    uint2 sv0 = make_uint2(0u, 0u);
    Job job;
    uint32_t n_map_tris = 0u;
    if (valid) {
        const uint4 head = __ldcg(reinterpret_cast<const uint4*>(blk));
        job = decode_job(P, id);
        n_map_tris = __ldg(&P.env_maps[job.e].n_tris);
        const bool ego_active = __ldg(&P.agents[(size_t)job.e * P.A + job.a].active) != 0u;
        const float* rx = P.rig.ray_x + (size_t)job.k * P.W + job.t.x0;
        const float* ry = P.rig.ray_y + (size_t)job.k * P.H + job.t.y0;
        s.ray_x[warp][lane] = __ldg(rx + lane); s.ray_x[warp][lane + 32] = __ldg(rx + lane + 32);
        s.ray_y[warp][lane] = __ldg(ry + lane); s.ray_y[warp][lane + 32] = __ldg(ry + lane + 32);
        if (lane == 0) {
            load_camera(s.cam[warp], P.cams[job.view], P.cam[job.k], P.W, P.H);
            TileRef tr;
            tr.pixel0 = job.view * ((size_t)P.H * P.W) + (size_t)job.t.y0 * P.W + job.t.x0;
            tr.bg_row0 = job.k * P.H + job.t.y0;
            tr.active = ego_active ? 1 : 0;
            s.tile[warp] = tr;
        }
        n_big = (int)(head.x & 0xffffu);
        ns = head.x == SURV_OVERFLOW ? -1 : n_big + (int)(head.x >> 16);
        if (ns > FPOOL) ns = -1;                            // more survivors than the whole pool
        // the first survivor of this lane (front list, then back list); the others are fetched in the set-up loop
        if (lane < ns) sv0 = __ldcg(blk + 2 + (lane < n_big ? lane : W_SURV - 1 - (lane - n_big)));
    }
    if (lane == 0) s.n_surv[warp] = ns;
#pragma unroll
    for (int i = 0; i < FSTRIP_KEYS / 2 / 32; ++i)
        reinterpret_cast<ulonglong2*>(s.key[warp])[i * 32 + lane] = make_ulonglong2(0ull, 0ull);
    __syncthreads();
    StripView sv;
    sv.key = s.key[warp];
    // Rounds: every thread lays the record pool out alike -- the tiles not yet rendered, in order,
    // as long as they fit.  One byte per tile: first record, and count (0xff: not in this round).
    uint32_t done = 0u;                                      // bit j: tile j is rendered, absent, or left to the cooperative kernel
#pragma unroll
    for (int j = 0; j < NW; ++j)
        if (s.n_surv[j] < 0) done |= 1u << j;
#pragma unroll 1
    while (done != (1u << NW) - 1u) {
        uint32_t bases = 0u, cnts = 0u, now = 0u;
        {
            int off = 0;
#pragma unroll
            for (int j = 0; j < NW; ++j) {
                const int c = s.n_surv[j];
                bases |= (uint32_t)off << (8 * j);
                if (!((done >> j) & 1u) && off + c <= FPOOL) { cnts |= (uint32_t)c << (8 * j); off += c; now |= 1u << j; }
                else cnts |= 0xffu << (8 * j);
            }
        }
        // ---- set-up by the tile's warp: survivor i becomes record i
        if ((now >> warp) & 1u) {
            const int my_base = (int)((bases >> (8 * warp)) & 0xffu);
            const int my_cnt = (stop == 14) ? 0 : ns;
            for (int i = lane; i < my_cnt; i += 32) {
                const uint2 svi = (i < 32) ? sv0 : __ldcg(blk + 2 + (i < n_big ? i : W_SURV - 1 - (i - n_big)));
                V3 V[4], Pn;
                uint32_t key_lo, flags;
                fetch_survivor(s.cam[warp], P, svi.x, job.e, n_map_tris, V, Pn, key_lo, flags);
                PrimEq q;
                if (!prim_equations(V, flags & 1u, flags, Pn, q)) { s.pool.box[my_base + i] = REC_DEAD; continue; }
                write_record(s.pool, my_base + i, q, key_lo, svi.y, (tiny_box(svi.y) ? REC_TINY : 0u) | (record_in_range(V, P) ? REC_INRANGE : 0u));
            }
        }
        if (threadIdx.x == 0) s.next_task = 0;
        __syncthreads();
        if (stop == 10) return;
        // ---- the strips of this round's tiles are tasks that the warps draw from a counter
#pragma unroll 1
        for (;;) {
            int task = 0;
            if (lane == 0) task = atomicAdd(&s.next_task, 1);
            task = __shfl_sync(0xffffffffu, task, 0);
            if (task >= NW * FSTRIPS) break;
            const int j = task / FSTRIPS, ys = (task % FSTRIPS) * FSTRIP;
            const int cj = (int)((cnts >> (8 * j)) & 0xffu);
            if (cj == 0xff) continue;
            const TileRef tr = s.tile[j];
            uint32_t bgc[2] = {P.cls_sky, P.cls_sky};
            float bgz[2] = {P.far_z, P.far_z};
            if (tr.active) {                                 // background of the rows this lane stores
                const uint32_t* bg_cls = P.rig.bg_cls + tr.bg_row0 + ys + (lane >> 2);
                const float* bg_z = P.rig.bg_z + tr.bg_row0 + ys + (lane >> 2);
                bgc[0] = __ldg(bg_cls); bgz[0] = __ldg(bg_z);
                if (FSTRIP == 16) { bgc[1] = __ldg(bg_cls + 8); bgz[1] = __ldg(bg_z + 8); }
            }
            sv.ray_x = s.ray_x[j]; sv.ray_y = s.ray_y[j] + ys;
            uint32_t touched = raster_strip_full(sv, s.pool, (int)((bases >> (8 * j)) & 0xffu), (stop == 14) ? 0 : cj, ys, P.w_near, P.w_far, stop, lane);
            if (stop == 5) touched = 0xffffu;
            if (stop == 6) touched |= 0x80000000u;
            const size_t o = tr.pixel0 + (size_t)ys * P.W;
            if (stop != 8) store_strip_full(sv.key, P.out_class + o, P.out_depth + o, P.W, touched, bgc, bgz, lane);
            __syncwarp();
        }
        done |= now;
        if (done != (1u << NW) - 1u) __syncthreads();        // the pool is reused by the next round
    }
    // ---- the rest: tiles with too many survivors, or whose cull lists overflowed, are left to the cooperative kernel
    if (threadIdx.x < NW && s.n_surv[threadIdx.x] == -1)
        P.overflow[1u + atomicAdd(&P.overflow[0], 1u)] = blockIdx.x * (unsigned)NW + threadIdx.x;
}

// The tiles the fused kernel left out, a CTA at a time.
template <class TL, bool FULL>
__global__ void __launch_bounds__(NTHREADS, 5) cooperative_kernel(const __grid_constant__ RenderParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TileSmem& cs = *reinterpret_cast<TileSmem*>(smem_raw);
    TL n = {};
    const unsigned count = __ldcg(&P.overflow[0]);
    for (unsigned i = blockIdx.x; i < count; i += gridDim.x) {
        cooperative_job<TL, FULL>(cs, P, __ldcg(&P.overflow[1u + i]), n);
        __syncthreads();
    }
    flush_counters(P, n);
}

#ifdef PIC_PROFILE
}  // namespace pic
#include <cstdlib>
namespace pic {
// profiling aid: extra dynamic shared memory per CTA lowers the number of resident CTAs per SM
static size_t smem_pad() { const char* e = getenv("PIC_SMEM_PAD"); return e ? (size_t)atoi(e) : 0; }
#define RENDER_SMEM (RENDER_SMEM_BASE + smem_pad())
#else
#define RENDER_SMEM RENDER_SMEM_BASE
#endif
#define FULL_SMEM (sizeof(FullSmem) + (RENDER_SMEM - RENDER_SMEM_BASE))
size_t render_smem_bytes() { return RENDER_SMEM; }

cudaError_t configure_render_kernel() {
    cudaError_t err = cudaFuncSetAttribute(render_full_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FULL_SMEM);
    if (err != cudaSuccess) return err;
    err = cudaFuncSetAttribute(render_kernel<NoTally, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)RENDER_SMEM);
    if (err != cudaSuccess) return err;
    err = cudaFuncSetAttribute(render_kernel<Tally, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)RENDER_SMEM);
    if (err != cudaSuccess) return err;
    err = cudaFuncSetAttribute(cooperative_kernel<NoTally, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TileSmem));
    if (err != cudaSuccess) return err;
    err = cudaFuncSetAttribute(cooperative_kernel<NoTally, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TileSmem));
    if (err != cudaSuccess) return err;
    return cudaFuncSetAttribute(cooperative_kernel<Tally, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TileSmem));
}

// ---------------------------------------------------------------------------------------------
// Coverage kernel (only with the occlusion option): for every tile and every other active agent,
// the pixels at which that agent's box, drawn alone, leaves a kept fragment.  A warp per tile;
// per agent, the six faces are rasterized into a bit mask of the tile (a lane per pixel of a face's
// pixel box), the set bits are counted and added to the view's count.  The arithmetic that decides
// a pixel is the production kernels' (pic_device.cuh).
// ---------------------------------------------------------------------------------------------
struct __align__(16) CoverWarp {
    float plane[6][4];
    float side[4][4];
    Cam cam;
    uint32_t mask[TILE * TILE / 32];
    float ray_x[TILE], ray_y[TILE];
};

__global__ void __launch_bounds__(NTHREADS) coverage_kernel(const __grid_constant__ RenderParams P) {
    __shared__ CoverWarp sm[NW];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned id = blockIdx.x * (unsigned)NW + warp;
    if (id >= P.n_jobs) return;
    CoverWarp& s = sm[warp];
    const Job job = decode_job(P, id);
    const TileCtx& t = job.t;
    const AgentGeom* env_agents = P.agents + (size_t)job.e * P.A;
    if (!env_agents[job.a].active) return;
    if (lane < 7) {
        Cam c;
        load_camera(c, P.cams[job.view], P.cam[job.k], P.W, P.H);
        if (lane == 6) s.cam = c;
        else tile_planes(s, lane, c, t);
    }
    for (int i = lane; i < TILE; i += 32) load_rays(s, P, job, i);
    for (int i = lane; i < TILE * TILE / 32; i += 32) s.mask[i] = 0u;
    __syncwarp();
    const Cam& c = s.cam;
    uint32_t* occ = P.occlusion + job.view * (size_t)P.A * 2u;
    for (int b = 0; b < P.A; ++b) {
        if (b == job.a) continue;
        const AgentGeom g = env_agents[b];
        if (!g.active || !box_faces(s, c, t, g)) continue;        // its bounding sphere misses the tile's frustum
        for (int f = 0; f < 6; ++f) {
            const uint32_t corners = face_corners(f);
            V3 V[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) V[q] = box_corner(c, g, (corners >> (4 * q)) & 7u);
            uint32_t box;
            if (!pixel_box(c, t, V, box)) continue;
            PrimEq q;
            if (!prim_equations(V, true, face_flags(corners), plane_normal(V, true), q)) continue;
            const int bx0 = box & 0xff, by0 = (box >> 8) & 0xff, bx1 = (box >> 16) & 0xff, by1 = box >> 24;
            const int w = bx1 - bx0 + 1, npx = w * (by1 - by0 + 1);
            for (int i = lane; i < npx; i += 32) {
                const int x = bx0 + i % w, y = by0 + i / w;
                if (fragment(q, s.ray_x[x], s.ray_y[y], t.w_near, t.w_far)) atomicOr(&s.mask[y * (TILE / 32) + (x >> 5)], 1u << (x & 31));
            }
        }
        __syncwarp();
        uint32_t cnt = 0u;
        for (int i = lane; i < TILE * TILE / 32; i += 32) { cnt += __popc(s.mask[i]); s.mask[i] = 0u; }
        cnt = __reduce_add_sync(0xffffffffu, cnt);
        if (lane == 0 && cnt) atomicAdd(occ + 2 * b + 1, cnt);
        __syncwarp();
    }
}

}  // namespace pic
#include "pic_coverage.cuh"
namespace pic {
#include "pic_colour.cuh"

size_t survivor_bytes_per_tile() { return sizeof(uint2) * SURV_STRIDE; }

cudaError_t launch_render_kernel(const RenderParams& P0, long long n_views, int sm_count, cudaStream_t stream) {
    RenderParams P = P0;
    const long long jobs = n_views * P.tiles_x * P.tiles_y;
    if (jobs > 0x7fffffffLL || (long long)P.E * P.A * P.K > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (jobs <= 0) return cudaSuccess;
    P.n_jobs = (uint32_t)jobs;
    const unsigned grid = (unsigned)((jobs + NW - 1) / NW);
    const bool full = P.W % TILE == 0 && P.H % TILE == 0 && P.out_depth32 == nullptr && P.occlusion == nullptr && (P.debug_flags & 15) == 0 &&
                      (reinterpret_cast<uintptr_t>(P.out_depth) & 31u) == 0;   // 256-bit depth stores
    // (a) cull: survivors per tile
    const unsigned cull_grid = (unsigned)((jobs + NW * CULL_ROUNDS - 1) / (NW * CULL_ROUNDS));
    if (P.counters) cull_kernel<Tally, false><<<cull_grid, NTHREADS, sizeof(CullSmem), stream>>>(P);
    else cull_kernel<NoTally, false><<<cull_grid, NTHREADS, sizeof(CullSmem), stream>>>(P);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    // (b)-(d) set-up, raster, store
    if (P.counters) render_kernel<Tally, false><<<grid, NTHREADS, RENDER_SMEM, stream>>>(P);
    else if (full) render_full_kernel<<<grid, NTHREADS, FULL_SMEM, stream>>>(P);
    else render_kernel<NoTally, false><<<grid, NTHREADS, RENDER_SMEM, stream>>>(P);
    err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    // the tiles left out (their number is only known on the device): one wave of CTAs walks the list
    const long long wave = (long long)(sm_count > 0 ? sm_count : 148) * 5;
    const unsigned cgrid = (unsigned)(jobs < wave ? jobs : wave);
    if (P.counters) cooperative_kernel<Tally, false><<<cgrid, NTHREADS, sizeof(TileSmem), stream>>>(P);
    else if (full) cooperative_kernel<NoTally, true><<<cgrid, NTHREADS, sizeof(TileSmem), stream>>>(P);
    else cooperative_kernel<NoTally, false><<<cgrid, NTHREADS, sizeof(TileSmem), stream>>>(P);
    err = cudaGetLastError();
    if (err != cudaSuccess || !P.occlusion) return err;
    coverage_kernel<<<grid, NTHREADS, 0, stream>>>(P);
    return cudaGetLastError();
}

// The coverage pass alone (after the exhaustive kernel, which counts the visible pixels itself).
cudaError_t launch_coverage_kernel(const RenderParams& P0, long long n_views, cudaStream_t stream) {
    RenderParams P = P0;
    const long long jobs = n_views * P.tiles_x * P.tiles_y;
    if (jobs <= 0 || !P.occlusion) return cudaSuccess;
    if (jobs > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    P.n_jobs = (uint32_t)jobs;
    coverage_kernel<<<(unsigned)((jobs + NW - 1) / NW), NTHREADS, 0, stream>>>(P);
    return cudaGetLastError();
}

}  // namespace pic
