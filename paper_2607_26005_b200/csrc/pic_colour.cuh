// Colour kernel (included by pic_render.cu, inside namespace pic): the paper's output format (Sec. 3.2) --
// 8-bit RGB images of flat-shaded primitives, box faces coloured per face with depth-aware brightness,
// optionally antialiased by analytic coverage at one sample per pixel.
//
// The paper gives neither colours nor a coverage formula; the definition implemented here is:
//   colour        a palette gives every class an RGB triple; a map primitive has its class's colour, face f of
//                 an agent's box its class's colour times FACE_SHADE[f] * (1 - 0.5 (z - near) / (far - near));
//   no AA         a pixel shows the nearest fragment that covers its centre (the class / depth image's winner);
//   AA            box filter over the pixel's unit square: a primitive's coverage is the exact area of the
//                 square inside all its edges and within the depth range of its plane; it leaves a fragment
//                 wherever that area is positive, at its plane's depth at the pixel centre (clamped to the
//                 range); a pixel's fragments are composited
//                 front to back, consecutive fragments of one surface (map primitives of one class; the faces of
//                 one box, of which only those turned towards the camera are drawn) first being merged into one
//                 layer: nearest first, each adds its coverage, and its colour with that weight, until the layer
//                 is full.
//
// Structure: the cull kernel's survivor lists (made with conservative pixel boxes when antialiasing) are set up
// into a record pool shared by the CTA's four tiles, in rounds like render_full_kernel; 8-row strips are tasks.
// A strip keeps, per pixel, the nearest FULLY covering fragment as a 64-bit key (unsigned max, as in the other
// kernels, with the record's slot in the low byte) and a linked list of the partially covering fragments in
// front of it (1/z, coverage in 14 bits, slot); the strip's warp owns both, so no atomics are needed.  The
// resolve walks each pixel's list in depth order, merges, composites and stores 16 pixels (48 bytes) per lane.
#pragma once

constexpr int CSTRIP = 8;                       // pixel rows of a strip
constexpr int CSTRIPS = TILE / CSTRIP;
constexpr int CSTRIP_KEYS = TILE * CSTRIP;
constexpr int CPOOL = 254;                      // records shared by the four tiles (a tile's survivors always fit: W_SURV < CPOOL)
constexpr int CFRAGS = 1023;                    // partially covering fragments of a strip (10-bit links, 0 ends a list)
constexpr uint32_t STATUS_COLOUR_INCOMPLETE = 2u;   // = PIC_FLAG_COLOUR_INCOMPLETE of the public header
constexpr uint32_t STATUS_COLOUR_FRAGMENTS = 4u;    // = PIC_FLAG_COLOUR_FRAGMENTS
static_assert(W_SURV <= CPOOL && CPOOL <= 256, "a tile's survivors fit the pool; a slot fits the key's low byte");

__constant__ float FACE_SHADE[6] = {0.60f, 1.00f, 0.70f, 0.85f, 0.40f, 0.92f};   // rear, front, right, left, bottom, top

struct __align__(16) ColourPool {
    float4 nx[CPOOL], ny[CPOOL], nz[CPOOL];     // edge functions E_i = nx[i] rx + ny[i] ry + nz[i]
    float4 w[CPOOL];                            // 1/z plane wx, wy, wz; key low word (index, class)
    uint32_t box[CPOOL];                        // pixel box (6 bits per coordinate), top-left bits << 24, REC_DEAD
    float shade[CPOOL];                         // box faces: the face's factor; map primitives: 0 (not shaded)
    uint32_t surface[CPOOL];                    // fragments of equal surface merge: a map primitive's class, 256 + agent of a box
};

struct __align__(16) ColourSmem {
    unsigned long long key[NW][CSTRIP_KEYS];    // warp w's strip: nearest fully covering fragment per pixel
    unsigned long long frag[NW][CFRAGS + 1];    // its partial fragments: bits(1/z) << 32 | coverage << 18 | slot << 10 | next
    uint16_t head[NW][CSTRIP_KEYS];             // first fragment of each pixel's list (0: none)
    ColourPool pool;
    float ray_x[NW][TILE], ray_y[NW][TILE];     // ray tables of tile w
    Cam cam[NW];
    Job job[NW];
    int active[NW];
    int n_surv[NW];
    int next_task;
};
static_assert(sizeof(ColourSmem) <= 74 * 1024, "three CTAs per SM");

struct RayView { float* ray_x; float* ray_y; };

// The six lines of a record at one pixel: values at the pixel centre (edges, 1/z - 1/far, 1/near - 1/z).
struct PixelLines { float e[CLINES]; };

// Coverage (14 bits) of one pixel by a record, given its lines at the pixel centre and their half ranges hh over
// the pixel (a line with e >= hh contains the whole pixel): the closed form if exactly one line crosses the pixel.
// Anything else (two or more lines: a strip, a vertex) returns COVERAGE_PENDING: those pixels are few per cell, so
// their areas are worked out later, a lane each (flush_pending) -- which is also less code in the cell loop, and the
// instruction cache is this kernel's bottleneck.
constexpr uint32_t COVERAGE_PENDING = 0x3fffu, COVERAGE_MAX = 0x3ffeu;
__device__ __forceinline__ uint32_t coverage14(const PixelLines& L, const PrimEq& q, const float (&hh)[CLINES], float du, float dv) {
    int n_part = 0;
    float e1 = 0.f, a1 = 0.f, b1 = 0.f;      // the line that crosses the pixel
#pragma unroll
    for (int i = 0; i < CLINES; ++i) {
        const float ai = (i < 4 ? q.nx[i] : i == 4 ? q.wx : -q.wx) * du, bi = (i < 4 ? q.ny[i] : i == 4 ? q.wy : -q.wy) * dv;
        if (L.e[i] < hh[i]) { ++n_part; e1 = L.e[i]; a1 = ai; b1 = bi; }
    }
    if (n_part != 1) return COVERAGE_PENDING;
    return min((uint32_t)(edge_coverage(e1, a1, b1) * 16383.f + 0.5f), COVERAGE_MAX);
}

// The strip's queue of pending pixels (pixel << 8 | slot; it grows down from the top of the fragment array while
// the lists grow up from its bottom), a lane each: the record's six lines at the pixel, the exact area, the depth;
// pixels with a positive area join their pixel's list.  The newest items -- those next to the lists' end -- go first,
// so the entries written never reach items not yet read.
__device__ __noinline__ void flush_pending(const unsigned long long* key, unsigned long long* frag, uint16_t* head, int& n_frag, int& n_pend, const ColourPool& pool,
                                              const float* ray_x, const float* ray_y, float du, float dv, float w_near, float w_far, int lane) {
    while (n_pend > 0) {
        const int take = min(n_pend, 32);
        const bool have = lane < take;
        const uint32_t item = have ? (uint32_t)frag[CFRAGS - (n_pend - 1) + lane] : 0u;
        __syncwarp();
        uint32_t a14 = 0u;
        float wc = 0.f;
        const uint32_t pix = item >> 8, slot = item & 0xffu;
        float area = 0.f;
        float e[CLINES], a[CLINES], b[CLINES];
        float w = 0.f;
#pragma unroll
        for (int j = 0; j < CLINES; ++j) { e[j] = 1.f; a[j] = 0.f; b[j] = 0.f; }
        if (have) {
            const float rx = ray_x[pix & (TILE - 1)], ry = ray_y[pix >> 6];
            const float4 r0 = pool.nx[slot], r1 = pool.ny[slot], r2 = pool.nz[slot], r3 = pool.w[slot];
            const float nx[4] = {r0.x, r0.y, r0.z, r0.w}, ny[4] = {r1.x, r1.y, r1.z, r1.w}, nz[4] = {r2.x, r2.y, r2.z, r2.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) { e[j] = fm(nx[j], rx, fm(ny[j], ry, nz[j])); a[j] = nx[j] * du; b[j] = ny[j] * dv; }
            w = fm(r3.x, rx, fm(r3.y, ry, r3.z));
            e[4] = w - w_far; e[5] = w_near - w; a[4] = r3.x * du; b[4] = r3.y * dv; a[5] = -a[4]; b[5] = -b[4];
            area = pixel_coverage<CLINES>(e, a, b);
        }
        if (have) {
            a14 = min((uint32_t)(area * 16383.f + 0.5f), COVERAGE_MAX);
            wc = fminf(fmaxf(w, w_far), w_near);
            // (only fragments in front of the pixel's nearest fully covering fragment so far are kept)
            if (!(make_key(__float_as_uint(wc), 0xffffffffu) > key[key_index((int)(pix & (TILE - 1)), (int)(pix >> 6))])) a14 = 0u;
        }
        n_pend -= take;
        // (two items of a round may belong to one pixel -- two records with a vertex there -- so the lists are
        // extended one lane after the other)
        const unsigned m = __ballot_sync(0xffffffffu, a14 != 0u);
        const int idx = n_frag + 1 + __popc(m & ((1u << lane) - 1u));
        // lanes whose pixel no other lane of the round shares link their entries at once
        const bool alone = __popc(__match_any_sync(0xffffffffu, a14 != 0u ? pix : 0x10000u + lane)) == 1;
        if (a14 != 0u && alone) {
            frag[idx] = ((unsigned long long)__float_as_uint(wc) << 32) | (a14 << 18) | (slot << 10) | head[pix];
            head[pix] = (uint16_t)idx;
        }
        for (unsigned rest = __ballot_sync(0xffffffffu, a14 != 0u && !alone); rest; rest &= rest - 1) {
            if (lane == __ffs(rest) - 1) {
                frag[idx] = ((unsigned long long)__float_as_uint(wc) << 32) | (a14 << 18) | (slot << 10) | head[pix];
                head[pix] = (uint16_t)idx;
            }
            __syncwarp();
        }
        n_frag += __popc(m);
    }
}

// A 16 x 4 pixel cell of a strip against one record; a lane handles two adjacent pixels.
template <bool AA>
__device__ __forceinline__ void colour_cell(unsigned long long* key, uint16_t* head, unsigned long long* frag, int& n_frag, int& n_pend, bool& dropped,
                                            const float* ray_x, const float* ray_y, const PrimEq& q, const float (&thr)[4],
                                            const float (&hh)[CLINES], float du, float dv, uint32_t key_lo, uint32_t slot,
                                            float w_near, float w_far, int xx, int yy, int row_lo, int row_hi, int col_lo, int col_hi, int lane) {
    const int x = xx + (lane & 7) * 2, y = yy + (lane >> 3);
    const float2 rx = *reinterpret_cast<const float2*>(ray_x + x);
    const float ry = ray_y[y];
    const float wt = fm(q.wy, ry, q.wz);
    const float w0 = fm(q.wx, rx.x, wt), w1 = fm(q.wx, rx.y, wt);
    PixelLines L0, L1;
    bool full0 = true, full1 = true, out0 = false, out1 = false;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float te = fm(q.ny[e], ry, q.nz[e]);
        L0.e[e] = fm(q.nx[e], rx.x, te); L1.e[e] = fm(q.nx[e], rx.y, te);
        if (!AA) { full0 = full0 && (L0.e[e] > thr[e]); full1 = full1 && (L1.e[e] > thr[e]); }
    }
    L0.e[4] = w0 - w_far; L0.e[5] = w_near - w0; L1.e[4] = w1 - w_far; L1.e[5] = w_near - w1;
    if (AA) {
#pragma unroll
        for (int e = 0; e < CLINES; ++e) {
            full0 = full0 && (L0.e[e] >= hh[e]); full1 = full1 && (L1.e[e] >= hh[e]);
            out0 = out0 || (L0.e[e] <= -hh[e]); out1 = out1 || (L1.e[e] <= -hh[e]);
        }
    } else {
        full0 = full0 && (w0 >= w_far) && (w0 <= w_near); full1 = full1 && (w1 >= w_far) && (w1 <= w_near);
    }
    unsigned long long* kp = key + key_index(x, y);
    const ulonglong2 kk = *reinterpret_cast<const ulonglong2*>(kp);
    // (a partially covered pixel's depth is its plane's at the pixel centre, clamped to the depth range)
    const float c0 = AA ? fminf(fmaxf(w0, w_far), w_near) : w0, c1 = AA ? fminf(fmaxf(w1, w_far), w_near) : w1;
    const unsigned long long k0 = make_key(__float_as_uint(c0), key_lo), k1 = make_key(__float_as_uint(c1), key_lo);
    if (full0 && k0 > kk.x) kp[0] = k0;
    if (full1 && k1 > kk.y) kp[1] = k1;
    if (AA) {
        // partially covered pixels in front of the nearest fully covering fragment seen so far
        const bool in_rows = y >= row_lo && y < row_hi;        // (lists are kept for a window of the strip's pixels at a time)
        bool push0 = in_rows && x >= col_lo && x < col_hi && !full0 && !out0 && k0 > kk.x;
        bool push1 = in_rows && x + 1 >= col_lo && x + 1 < col_hi && !full1 && !out1 && k1 > kk.y;
        if (__any_sync(0xffffffffu, push0 || push1)) {
            // (one copy of the coverage code serves both pixels: the instruction cache matters more than the selects)
            uint32_t a0 = 0u, a1 = 0u;
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                PixelLines L;
#pragma unroll
                for (int e = 0; e < CLINES; ++e) L.e[e] = h ? L1.e[e] : L0.e[e];
                const uint32_t av = (h ? push1 : push0) ? coverage14(L, q, hh, du, dv) : 0u;
                if (h) a1 = av; else a0 = av;
            }
            const bool pend0 = push0 && a0 == COVERAGE_PENDING, pend1 = push1 && a1 == COVERAGE_PENDING;
            push0 = push0 && a0 != 0u && !pend0; push1 = push1 && a1 != 0u && !pend1;
            const unsigned m0 = __ballot_sync(0xffffffffu, push0), m1 = __ballot_sync(0xffffffffu, push1);
            const unsigned q0 = __ballot_sync(0xffffffffu, pend0), q1 = __ballot_sync(0xffffffffu, pend1);
            const unsigned below = (1u << lane) - 1u;
            const int pix = y * TILE + x;
            // room: lists and queue share the array; what does not fit is dropped (and the call says so)
            const bool room = n_frag + n_pend + __popc(m0) + __popc(m1) + __popc(q0) + __popc(q1) <= CFRAGS;
            if (room) {
                const int i0 = n_frag + 1 + __popc(m0 & below), i1 = n_frag + 1 + __popc(m0) + __popc(m1 & below);
                if (push0) { frag[i0] = ((unsigned long long)__float_as_uint(c0) << 32) | (a0 << 18) | (slot << 10) | head[pix]; head[pix] = (uint16_t)i0; }
                if (push1) { frag[i1] = ((unsigned long long)__float_as_uint(c1) << 32) | (a1 << 18) | (slot << 10) | head[pix + 1]; head[pix + 1] = (uint16_t)i1; }
                n_frag += __popc(m0) + __popc(m1);
                if (pend0) frag[CFRAGS - (n_pend + __popc(q0 & below))] = ((uint32_t)pix << 8) | slot;
                if (pend1) frag[CFRAGS - (n_pend + __popc(q0) + __popc(q1 & below))] = ((uint32_t)(pix + 1) << 8) | slot;
                n_pend += __popc(q0) + __popc(q1);
            } else {
                dropped = true;
            }
        }
    }
}

// Colour of a fragment of the record in `slot` at reciprocal depth w.
__device__ __forceinline__ void shade_fragment(const ColourPool& pool, const RenderParams& P, uint32_t slot, float w, float& r, float& g, float& b) {
    const uint32_t cls = __float_as_uint(pool.w[slot].w) & 0xffu;
    const float sh = pool.shade[slot];
    float k = 1.f;
    if (sh > 0.f) k = sh * (1.f - 0.5f * __fdividef(__fdividef(1.f, w) - P.near_z, P.far_z - P.near_z));
    const uint8_t* pal = P.palette + 3u * cls;
    r = k * (float)__ldg(pal); g = k * (float)__ldg(pal + 1); b = k * (float)__ldg(pal + 2);
}

// Colour of a pixel with a list of partially covering fragments: front to back, the list's fragments in front of the
// fully covering one `k`, then that one, then the background.  Consecutive fragments of one surface form a layer:
// each adds its coverage until the layer is full.  Returns the colour packed 8 bits per channel.
__device__ __forceinline__ uint32_t composite_pixel(unsigned long long k, uint32_t hd, const unsigned long long* frag, const ColourPool& pool,
                                                    const RenderParams& P, float bgr, float bgg, float bgb) {
    const uint32_t w_opq = (uint32_t)(k >> 32);
    float T = 1.f, acc = 0.f, R = 0.f, G = 0.f, B = 0.f;
    uint32_t cur = 0xffffffffu;
    unsigned long long prev = ~0ull;
    for (int it = 0; it < 64 && T > 0.f; ++it) {
        // the nearest remaining fragment: the largest (1/z, entry) below the last one taken; at the end, the opaque one
        unsigned long long best = 0ull;
        uint32_t best_lo = 0u;
        for (uint32_t i = hd; i;) {
            const unsigned long long en = frag[i];
            const unsigned long long cand = (en & 0xffffffff00000000ull) | i;
            if (cand < prev && cand > best && (uint32_t)(en >> 32) > w_opq) { best = cand; best_lo = (uint32_t)en; }
            i = (uint32_t)en & 1023u;
        }
        uint32_t slot, wb;
        float alpha;
        if (best) { prev = best; slot = (best_lo >> 10) & 0xffu; alpha = (float)((best_lo >> 18) & 0x3fffu) * (1.f / 16383.f); wb = (uint32_t)(best >> 32); }
        else if (k && prev != 0ull) { prev = 0ull; slot = (uint32_t)k & 0xffu; alpha = 1.f; wb = w_opq; }
        else break;
        const uint32_t surf = pool.surface[slot];
        if (surf != cur) { T *= 1.f - acc; cur = surf; acc = 0.f; }
        const float add = fminf(alpha, 1.f - acc) * T;
        float cr, cg, cb;
        shade_fragment(pool, P, slot, __uint_as_float(wb), cr, cg, cb);
        R = fm(add, cr, R); G = fm(add, cg, G); B = fm(add, cb, B);
        acc += fminf(alpha, 1.f - acc);
    }
    T *= 1.f - acc;
    R = fm(T, bgr, R); G = fm(T, bgg, G); B = fm(T, bgb, B);
    return (uint32_t)fminf(fmaxf(R + 0.5f, 0.f), 255.f) | ((uint32_t)fminf(fmaxf(G + 0.5f, 0.f), 255.f) << 8) |
           ((uint32_t)fminf(fmaxf(B + 0.5f, 0.f), 255.f) << 16);
}

constexpr unsigned long long KEY_RESOLVED = 1ull << 63;     // (a key's high word is the bits of a positive float: bit 63 is free)

// Rows of a strip of tile `jb` -> colours: the pixels that have a list are composited, lane l taking pixels l, l + 32, ...
// so that a row crowded with fragments (the horizon) is shared by all lanes; their colour replaces the pixel's key
// (composite_rows).  At the end every lane converts 16 consecutive pixels of a row, resets what it reads, and stores
// (resolve_store_colour).
__device__ __forceinline__ void composite_rows(unsigned long long* key, uint16_t* head, const unsigned long long* frag,
                                               const ColourPool& pool, const RenderParams& P, const Job& jb, bool ego_active,
                                               int ys, int row_lo, int row_hi, int lane) {
    {
#pragma unroll 1
        for (int i = row_lo * (TILE / 32); i < row_hi * (TILE / 32); ++i) {
            const int p = i * 32 + lane, x = p & (TILE - 1), y = p >> 6;
            const uint32_t hd = head[p];
            if (hd) {
                head[p] = 0;
                const int gy = jb.t.y0 + ys + y;
                uint32_t bgc = P.cls_sky;
                if (ego_active && gy < P.H) bgc = __ldg(P.rig.bg_cls + (size_t)jb.k * P.H + gy);
                unsigned long long* kp = key + key_index(x, y);
                *kp = KEY_RESOLVED | composite_pixel(*kp, hd, frag, pool, P, (float)__ldg(P.palette + 3u * bgc), (float)__ldg(P.palette + 3u * bgc + 1),
                                                     (float)__ldg(P.palette + 3u * bgc + 2));
            }
        }
        __syncwarp();
    }
}

// (the same with all 16 pixels of a lane unrolled and three 128-bit stores: faster where the kernel's code is small
// enough anyway -- the plain instantiation)
__device__ __forceinline__ void resolve_store_wide(unsigned long long* key, const ColourPool& pool, const RenderParams& P, const Job& jb,
                                                     bool ego_active, int ys, bool vec_ok, int lane) {
    const int y = lane >> 2, xs = (lane & 3) * 16;
    const int gy = jb.t.y0 + ys + y;
    uint32_t bgc = P.cls_sky;
    if (ego_active && gy < P.H) bgc = __ldg(P.rig.bg_cls + (size_t)jb.k * P.H + gy);
    const uint32_t bg8 = (uint32_t)__ldg(P.palette + 3u * bgc) | ((uint32_t)__ldg(P.palette + 3u * bgc + 1) << 8) | ((uint32_t)__ldg(P.palette + 3u * bgc + 2) << 16);
    uint32_t ow[12];
#pragma unroll
    for (int i = 0; i < 12; ++i) ow[i] = 0u;
#pragma unroll
    for (int j = 0; j < 16; j += 2) {
        ulonglong2* kp = reinterpret_cast<ulonglong2*>(key + key_index(xs + j, y));
        const ulonglong2 kk = *kp;
        *kp = make_ulonglong2(0ull, 0ull);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const unsigned long long k = h ? kk.y : kk.x;
            uint32_t c = bg8;
            if (k & KEY_RESOLVED) c = (uint32_t)k & 0xffffffu;
            else if (k) {
                float R, G, B;
                shade_fragment(pool, P, (uint32_t)k & 0xffu, __uint_as_float((uint32_t)(k >> 32)), R, G, B);
                c = (uint32_t)fminf(R + 0.5f, 255.f) | ((uint32_t)fminf(G + 0.5f, 255.f) << 8) | ((uint32_t)fminf(B + 0.5f, 255.f) << 16);
            }
            const int n = 3 * (j + h);           // byte offset of the pixel in the lane's 48 bytes
            ow[n >> 2] |= c << (8 * (n & 3));
            if ((n & 3) > 1) ow[(n >> 2) + 1] |= c >> (8 * (4 - (n & 3)));
        }
    }
    if (ys + y >= jb.t.th || xs >= jb.t.tw) return;
    uint8_t* dst = P.out_rgb + 3u * ((jb.view * (size_t)P.H + gy) * (size_t)P.W + jb.t.x0 + xs);
    if (vec_ok && xs + 16 <= jb.t.tw) {
        uint4* d4 = reinterpret_cast<uint4*>(dst);
        d4[0] = make_uint4(ow[0], ow[1], ow[2], ow[3]);
        d4[1] = make_uint4(ow[4], ow[5], ow[6], ow[7]);
        d4[2] = make_uint4(ow[8], ow[9], ow[10], ow[11]);
    } else {
#pragma unroll
        for (int n = 0; n < 48; ++n)
            if (n / 3 + xs < jb.t.tw) dst[n] = (uint8_t)(ow[n >> 2] >> (8 * (n & 3)));
    }
}

__device__ __forceinline__ void resolve_store_colour(unsigned long long* key, const ColourPool& pool, const RenderParams& P, const Job& jb,
                                                     bool ego_active, int ys, bool vec_ok, int lane) {
    const int y = lane >> 2, xs = (lane & 3) * 16;
    const int gy = jb.t.y0 + ys + y;
    uint32_t bgc = P.cls_sky;
    if (ego_active && gy < P.H) bgc = __ldg(P.rig.bg_cls + (size_t)jb.k * P.H + gy);
    const uint32_t bg8 = (uint32_t)__ldg(P.palette + 3u * bgc) | ((uint32_t)__ldg(P.palette + 3u * bgc + 1) << 8) | ((uint32_t)__ldg(P.palette + 3u * bgc + 2) << 16);
    const bool row_ok = ys + y < jb.t.th;
    uint8_t* dst = P.out_rgb + 3u * ((jb.view * (size_t)P.H + gy) * (size_t)P.W + jb.t.x0 + xs);
    // four groups of four pixels (12 bytes, three words) each; the loop is not unrolled: one copy of the shading code
#pragma unroll 1
    for (int g = 0; g < 4; ++g) {
        uint32_t ow[3] = {0u, 0u, 0u};
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
            ulonglong2* kp = reinterpret_cast<ulonglong2*>(key + key_index(xs + 4 * g + 2 * h2, y));
            const ulonglong2 kk = *kp;
            *kp = make_ulonglong2(0ull, 0ull);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const unsigned long long k = h ? kk.y : kk.x;
                uint32_t c = bg8;
                if (k & KEY_RESOLVED) c = (uint32_t)k & 0xffffffu;
                else if (k) {
                    float R, G, B;
                    shade_fragment(pool, P, (uint32_t)k & 0xffu, __uint_as_float((uint32_t)(k >> 32)), R, G, B);
                    c = (uint32_t)fminf(R + 0.5f, 255.f) | ((uint32_t)fminf(G + 0.5f, 255.f) << 8) | ((uint32_t)fminf(B + 0.5f, 255.f) << 16);
                }
                const int n = 3 * (2 * h2 + h);      // byte offset of the pixel in the group's 12 bytes
                ow[n >> 2] |= c << (8 * (n & 3));
                if ((n & 3) > 1) ow[(n >> 2) + 1] |= c >> (8 * (4 - (n & 3)));
            }
        }
        const int x = xs + 4 * g;
        if (row_ok && x < jb.t.tw) {
            if (vec_ok && x + 4 <= jb.t.tw) {
                uint32_t* d32 = reinterpret_cast<uint32_t*>(dst + 12 * g);
                d32[0] = ow[0]; d32[1] = ow[1]; d32[2] = ow[2];
            } else {
#pragma unroll
                for (int n = 0; n < 12; ++n)
                    if (n / 3 + x < jb.t.tw) dst[12 * g + n] = (uint8_t)(ow[n >> 2] >> (8 * (n & 3)));
            }
        }
    }
}

template <bool AA>
__global__ void __launch_bounds__(NTHREADS, 3) colour_kernel(const __grid_constant__ RenderParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    ColourSmem& s = *reinterpret_cast<ColourSmem*>(smem_raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned id = blockIdx.x * (unsigned)NW + warp;
    const bool valid = id < P.n_jobs;
    const uint2* blk = P.surv + (size_t)id * SURV_STRIDE;
    int ns = -2, n_big = 0;
    Job job;
    uint32_t n_map_tris = 0u;
    if (valid) {
        const uint4 head = __ldcg(reinterpret_cast<const uint4*>(blk));
        job = decode_job(P, id);
        n_map_tris = __ldg(&P.env_maps[job.e].n_tris);
        const bool ego_active = __ldg(&P.agents[(size_t)job.e * P.A + job.a].active) != 0u;
        RayView rv = {s.ray_x[warp], s.ray_y[warp]};
        load_rays(rv, P, job, lane); load_rays(rv, P, job, lane + 32);
        if (lane == 0) {
            load_camera(s.cam[warp], P.cams[job.view], P.cam[job.k], P.W, P.H);
            s.job[warp] = job;
            s.active[warp] = ego_active ? 1 : 0;
        }
        n_big = (int)(head.x & 0xffffu);
        ns = n_big + (int)(head.x >> 16);
        if (head.x == SURV_OVERFLOW) {
            // more visible primitives than the tile's list holds: the tile shows only the background, and the call says so
            ns = 0; n_big = 0;
            if (lane == 0) atomicOr(P.status, STATUS_COLOUR_INCOMPLETE);
        }
    }
    if (lane == 0) s.n_surv[warp] = ns;
#pragma unroll
    for (int i = 0; i < CSTRIP_KEYS / 2 / 32; ++i)
        reinterpret_cast<ulonglong2*>(s.key[warp])[i * 32 + lane] = make_ulonglong2(0ull, 0ull);
#pragma unroll
    for (int i = 0; i < CSTRIP_KEYS / 8 / 32; ++i)
        reinterpret_cast<uint4*>(s.head[warp])[i * 32 + lane] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    const bool vec_ok = (P.W % 16 == 0) && ((reinterpret_cast<uintptr_t>(P.out_rgb) & 15u) == 0);
    uint32_t done = 0u;
#pragma unroll
    for (int j = 0; j < NW; ++j)
        if (s.n_surv[j] < 0) done |= 1u << j;
#pragma unroll 1
    while (done != (1u << NW) - 1u) {
        // this round's tiles: those not yet rendered, in order, as long as their survivors fit the pool
        uint32_t bases = 0u, cnts = 0u, now = 0u;
        {
            int off = 0;
#pragma unroll
            for (int j = 0; j < NW; ++j) {
                const int c = s.n_surv[j];
                bases |= (uint32_t)off << (8 * j);
                if (!((done >> j) & 1u) && off + c <= CPOOL) { cnts |= (uint32_t)c << (8 * j); off += c; now |= 1u << j; }
                else cnts |= 0xffu << (8 * j);
            }
        }
        // ---- set-up by the tile's warp: survivor i becomes record base + i
        if ((now >> warp) & 1u) {
            const int my_base = (int)((bases >> (8 * warp)) & 0xffu);
            const Cam& c = s.cam[warp];
            for (int i = lane; i < ns; i += 32) {
                const uint2 svi = __ldcg(blk + 2 + (i < n_big ? i : W_SURV - 1 - (i - n_big)));
                V3 V[4], Pn;
                uint32_t key_lo, flags;
                fetch_survivor(c, P, svi.x, job.e, n_map_tris, V, Pn, key_lo, flags);
                float shade = 0.f;
                uint32_t surface = key_lo & 0xffu;
                bool drop = false;
                if (svi.x & SURV_FACE) {
                    const uint32_t b = (svi.x & ~SURV_FACE) >> 3, f = svi.x & 7u;
                    shade = FACE_SHADE[f];
                    surface = 256u + b;
                    if (AA) {
                        // faces whose outer side is turned away from the camera centre are not drawn: the camera
                        // centre (the origin) and the box's centre lie on the same side of the face's plane
                        const AgentGeom g = P.agents[(size_t)job.e * P.A + b];
                        const V3 bc = rotate_to_camera(c, sub(sub(g.x, c.px), c.mwx), sub(sub(g.y, c.py), c.mwy), sub(0.5f * g.h, c.mwz));
                        const float s_cam = -vdot(Pn, V[0]), s_box = vdot(Pn, vsub(bc, V[0]));
                        drop = !(s_cam * s_box < 0.f);
                    }
                }
                PrimEq q;
                const int slot = my_base + i;
                if (drop || !prim_equations(V, flags & 1u, flags, Pn, q)) { s.pool.box[slot] = REC_DEAD; continue; }
                const uint32_t box = svi.y;
                const uint32_t bx0 = box & 0xff, by0 = (box >> 8) & 0xff, bx1 = (box >> 16) & 0xff, by1 = box >> 24;
                s.pool.nx[slot] = make_float4(q.nx[0], q.nx[1], q.nx[2], q.nx[3]);
                s.pool.ny[slot] = make_float4(q.ny[0], q.ny[1], q.ny[2], q.ny[3]);
                s.pool.nz[slot] = make_float4(q.nz[0], q.nz[1], q.nz[2], q.nz[3]);
                s.pool.w[slot] = make_float4(q.wx, q.wy, q.wz, __uint_as_float(key_lo));
                s.pool.box[slot] = bx0 | (by0 << 6) | (bx1 << 12) | (by1 << 18) | (q.tl << 24);
                s.pool.shade[slot] = shade;
                s.pool.surface[slot] = surface;
            }
        }
        if (threadIdx.x == 0) s.next_task = 0;
        __syncthreads();
        // ---- the strips of this round's tiles are tasks that the warps draw from a counter
        unsigned long long* key = s.key[warp];
        uint16_t* head = s.head[warp];
        unsigned long long* frag = s.frag[warp];
#pragma unroll 1
        for (;;) {
            int task = 0;
            if (lane == 0) task = atomicAdd(&s.next_task, 1);
            task = __shfl_sync(0xffffffffu, task, 0);
            if (task >= NW * CSTRIPS) break;
            const int j = task / CSTRIPS, ys = (task % CSTRIPS) * CSTRIP;
            const int cj = (int)((cnts >> (8 * j)) & 0xffu);
            if (cj == 0xff) continue;
            const Job jb = s.job[j];
            if (ys >= jb.t.th) continue;
            const int first = (int)((bases >> (8 * j)) & 0xffu);
            const float* ray_x = s.ray_x[j];
            const float* ray_y = s.ray_y[j] + ys;
            const float du = __fdividef(1.f, s.cam[j].focx), dv = __fdividef(1.f, s.cam[j].focy);
            // The lists of partially covering fragments are kept for a window of the strip's rows at a time: all eight,
            // or, when the fragment array overflows (a dense soup of edges), half as many, again and again down to one
            // row -- the window is rasterized anew, the rows before it keep their composited colours (parked in their
            // keys, which no fragment can replace).  Before the first such retry the strip is rasterized once with an
            // empty window: that leaves every pixel's nearest fully covering fragment in its key, so the retries keep
            // only the fragments in front of it (in a soup, few).  A single row that still overflows (many coplanar
            // primitives cut by the near plane along it) is taken half as many columns at a time, down to one pixel.
            int win = CSTRIP, cw = TILE, row_next = 0, col_next = 0;
            bool prepass = false, prepass_done = false;
            while (row_next < CSTRIP) {
            const int row_lo = prepass ? 0 : row_next, row_hi = prepass ? 0 : min(row_next + win, CSTRIP);
            const int col_lo = col_next, col_hi = col_next + cw;
            int n_frag = 0, n_pend = 0;
            bool dropped = false;
            for (int base = 0; base < cj; base += 32) {
                uint32_t bw_lane = 0u;
                bool hit = false;
                if (base + lane < cj) {
                    bw_lane = s.pool.box[first + base + lane];
                    const int by0 = (bw_lane >> 6) & 63, by1 = (bw_lane >> 18) & 63;
                    hit = !(bw_lane & REC_DEAD) && by1 >= ys && by0 < ys + CSTRIP;
                }
                if (AA) {
                    // records whose pixel box is at most 4 x 4: every pixel of the box (in this strip's window) is queued as
                    // a (pixel, record) pair and worked off with the other pending pixels, a lane each -- far cheaper
                    // than walking a 64-pixel cell per record for the handful of pixels a distant primitive touches
                    const int bx0 = bw_lane & 63, bx1 = (bw_lane >> 12) & 63, by0 = (bw_lane >> 6) & 63, by1 = (bw_lane >> 18) & 63;
                    const bool small = hit && bx1 - bx0 < 4 && by1 - by0 < 4;
                    hit = hit && !small;
                    const int x0 = max(bx0, col_lo), x1 = min(bx1, col_hi - 1);
                    const int w = max(x1 - x0 + 1, 0), y0 = max(by0 - ys, row_lo), y1 = min(by1 - ys, row_hi - 1);
                    const int cnt = small ? w * max(y1 - y0 + 1, 0) : 0;
                    if (__any_sync(0xffffffffu, cnt > 0)) {
                        int incl = cnt;
#pragma unroll
                        for (int d = 1; d < 32; d <<= 1) {
                            const int up = __shfl_up_sync(0xffffffffu, incl, d);
                            if (lane >= d) incl += up;
                        }
                        const int total = __shfl_sync(0xffffffffu, incl, 31);
                        if (n_frag + n_pend + total <= CFRAGS) {
                            const uint32_t slot = (uint32_t)(first + base + lane);
                            for (int k = 0; k < cnt; ++k) {
                                const uint32_t pix = (uint32_t)((y0 + k / w) * TILE + x0 + k % w);
                                frag[CFRAGS - (n_pend + (incl - cnt) + k)] = (pix << 8) | slot;
                            }
                            n_pend += total;
                        } else {
                            dropped = true;
                        }
                        __syncwarp();
                        if (n_pend >= 96) flush_pending(key, frag, head, n_frag, n_pend, s.pool, ray_x, ray_y, du, dv, P.w_near, P.w_far, lane);
                    }
                }
                for (unsigned hits = __ballot_sync(0xffffffffu, hit); hits; hits &= hits - 1) {
                    const int src = __ffs(hits) - 1;
                    const uint32_t bw = __shfl_sync(0xffffffffu, bw_lane, src);
                    const int by0 = (bw >> 6) & 63, by1 = (bw >> 18) & 63, bx0 = bw & 63, bx1 = (bw >> 12) & 63;
                    const int ly0 = max(by0, ys) - ys, ly1 = min(by1, ys + CSTRIP - 1) - ys;
                    const uint32_t slot = (uint32_t)(first + base + src);
                    const float4 r0 = s.pool.nx[slot], r1 = s.pool.ny[slot], r2 = s.pool.nz[slot], r3 = s.pool.w[slot];
                    PrimEq q;
                    q.nx[0] = r0.x; q.nx[1] = r0.y; q.nx[2] = r0.z; q.nx[3] = r0.w;
                    q.ny[0] = r1.x; q.ny[1] = r1.y; q.ny[2] = r1.z; q.ny[3] = r1.w;
                    q.nz[0] = r2.x; q.nz[1] = r2.y; q.nz[2] = r2.z; q.nz[3] = r2.w;
                    q.wx = r3.x; q.wy = r3.y; q.wz = r3.z;
                    q.tl = (bw >> 24) & 15u;
                    const uint32_t key_lo = (__float_as_uint(r3.w) & 0xffffff00u) | slot;
                    float thr[4], hh[CLINES];
                    edge_thresholds(q.tl, thr);
#pragma unroll
                    for (int e = 0; e < 4; ++e) hh[e] = 0.5f * (fabsf(q.nx[e]) * du + fabsf(q.ny[e]) * dv);
                    hh[4] = hh[5] = 0.5f * (fabsf(q.wx) * du + fabsf(q.wy) * dv);
                    for (int yy = ly0 & ~3; yy <= ly1; yy += 4)
                        for (int xx = bx0 & ~15; xx <= bx1; xx += 16)
                            colour_cell<AA>(key, head, frag, n_frag, n_pend, dropped, ray_x, ray_y, q, thr, hh, du, dv, key_lo, slot, P.w_near, P.w_far, xx, yy, row_lo, row_hi, col_lo, col_hi, lane);
                    // the queue is worked off when it holds a few rounds' worth (working it off frees room only for the
                    // pixels whose area turns out to be zero, so a nearly full array is no reason to do it earlier)
                    if (AA && n_pend >= 96) {
                        __syncwarp();
                        flush_pending(key, frag, head, n_frag, n_pend, s.pool, ray_x, ray_y, du, dv, P.w_near, P.w_far, lane);
                    }
                }
                __syncwarp();
            }
            if (AA) flush_pending(key, frag, head, n_frag, n_pend, s.pool, ray_x, ray_y, du, dv, P.w_near, P.w_far, lane);
            __syncwarp();
            if (AA && prepass) { prepass = false; prepass_done = true; continue; }
            if (AA && dropped && (!prepass_done || win > 1 || cw > 1)) {    // too many fragments: this window again
                for (int p = row_lo * TILE + lane; p < row_hi * TILE; p += 32)
                    if ((p & (TILE - 1)) >= col_lo) head[p] = 0;  // (the columns before the window are done: their heads are 0)
                __syncwarp();
                if (!prepass_done) prepass = true;                // ... after the keys have been completed,
                else if (win > 1) win >>= 1;                      // ... then with half as many rows,
                else cw >>= 1;                                    // ... then with half as many columns of the one row
                continue;
            }
            if (AA && dropped && lane == 0) atomicOr(P.status, STATUS_COLOUR_FRAGMENTS);   // (more than 1 023 in front of the opaque surface of one pixel)
            if (AA) composite_rows(key, head, frag, s.pool, P, jb, s.active[j] != 0, ys, row_lo, row_hi, lane);
            col_next += cw;
            if (col_next >= TILE) { col_next = 0; row_next = row_hi; }
            }   // (windows)
            __syncwarp();
            if (AA) resolve_store_colour(key, s.pool, P, jb, s.active[j] != 0, ys, vec_ok, lane);
            else resolve_store_wide(key, s.pool, P, jb, s.active[j] != 0, ys, vec_ok, lane);
            __syncwarp();
        }
        done |= now;
        if (done != (1u << NW) - 1u) __syncthreads();        // the pool is reused by the next round
    }
}

cudaError_t configure_colour_kernel() {
    cudaError_t err = cudaFuncSetAttribute(colour_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ColourSmem));
    if (err != cudaSuccess) return err;
    return cudaFuncSetAttribute(colour_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ColourSmem));
}

// Colour images of n_views views: the cull kernel (conservative pixel boxes when antialiasing), then the colour kernel.
cudaError_t launch_colour_kernel(const RenderParams& P0, long long n_views, bool antialias, cudaStream_t stream) {
    RenderParams P = P0;
    const long long jobs = n_views * P.tiles_x * P.tiles_y;
    if (jobs > 0x7fffffffLL || (long long)P.E * P.A * P.K > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (jobs <= 0) return cudaSuccess;
    P.n_jobs = (uint32_t)jobs;
    P.debug_flags = 0;
    P.counters = nullptr;
    const unsigned grid = (unsigned)((jobs + NW - 1) / NW);
    if (antialias) cull_kernel<NoTally, true><<<grid, NTHREADS, sizeof(CullSmem), stream>>>(P);
    else cull_kernel<NoTally, false><<<grid, NTHREADS, sizeof(CullSmem), stream>>>(P);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    if (antialias) colour_kernel<true><<<grid, NTHREADS, sizeof(ColourSmem), stream>>>(P);
    else colour_kernel<false><<<grid, NTHREADS, sizeof(ColourSmem), stream>>>(P);
    return cudaGetLastError();
}
