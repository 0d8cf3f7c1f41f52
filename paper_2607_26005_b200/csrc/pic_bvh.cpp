// Host-side construction of the per-map culling hierarchy (runs once, in pic_scene_create).
//
// Input triangles are first fused pairwise into planar convex quads where the input allows it
// (two consecutive triangles of one class sharing an edge: road, marking and wall quads), then
// sorted along a Morton curve and cut into leaves of up to LEAF_PRIMS primitives; leaves are
// grouped by GROUP_LEAVES.  Primitives much longer than the average get leaves of their own, so
// that one long road quad does not inflate the box of its neighbouring lane markings.  The renderer tests group boxes, then
// leaf boxes, then primitives against each view frustum.
//
// The cull kernel uses a second, flatter structure over the same primitives: a uniform grid on
// the ground plane.  A primitive whose box (xy) has a half-diagonal of at most half a cell is
// "small" and is listed under the cell that holds the centre of its box; a second copy of the
// primitives is stored in that order, cell after cell, row-major, so the small primitives of a run
// of cells of one grid row are one contiguous range of it (the large ones follow, leaf by leaf).
// A view then needs one range per grid row that its frustum's footprint (widened by the largest
// half-diagonal of a small primitive) crosses.  The few primitives too large for a cell (long road
// quads) are kept in leaves of LARGE_LEAF_PRIMS with boxes, tested one by one.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <vector>

#include "pic_types.h"

namespace pic {

struct HostHierarchy {
    std::vector<Prim> prims;
    std::vector<Node> leaves;
    std::vector<Node> groups;
    std::vector<MapInfo> maps;
    std::vector<uint32_t> cell_start;
    std::vector<Prim> grid_prims;             // the same primitives once more, in grid order
    std::vector<Node> large_leaves;
};

namespace {

struct D3 { double x, y, z; };
inline D3 sub(D3 a, D3 b) { return {a.x - b.x, a.y - b.y, a.z - b.z}; }
inline D3 cross(D3 a, D3 b) { return {a.y * b.z - a.z * b.y, a.z * b.x - a.x * b.z, a.x * b.y - a.y * b.x}; }
inline double dot(D3 a, D3 b) { return a.x * b.x + a.y * b.y + a.z * b.z; }
inline double norm(D3 a) { return std::sqrt(dot(a, a)); }

struct F3 { float x, y, z; };
inline bool same(F3 a, F3 b) { return a.x == b.x && a.y == b.y && a.z == b.z; }
inline D3 d3(F3 a) { return {a.x, a.y, a.z}; }
inline bool lex_less(F3 a, F3 b) {
    if (a.x != b.x) return a.x < b.x;
    if (a.y != b.y) return a.y < b.y;
    return a.z < b.z;
}

// Try to fuse triangles a and b into the convex planar quad (q[0..3] in perimeter order).
bool fuse_quad(const F3 a[3], const F3 b[3], F3 q[4]) {
    for (int i = 0; i < 3; ++i) {
        // candidate: a's vertex i is the one b does not share
        F3 pa = a[i], s0 = a[(i + 1) % 3], s1 = a[(i + 2) % 3];
        int j0 = -1, j1 = -1;
        for (int j = 0; j < 3; ++j) {
            if (same(b[j], s0)) j0 = j;
            if (same(b[j], s1)) j1 = j;
        }
        if (j0 < 0 || j1 < 0 || j0 == j1) continue;
        F3 pb = b[3 - j0 - j1];
        if (same(pb, pa) || same(pb, s0) || same(pb, s1)) return false;
        D3 P[4] = {d3(pa), d3(s0), d3(pb), d3(s1)};
        D3 n = cross(sub(P[2], P[0]), sub(P[3], P[1]));
        double nn = norm(n);
        if (nn == 0.0) return false;
        // coplanar: the two diagonals' common normal must be orthogonal to every side
        double scale = 0.0;
        for (int k = 0; k < 4; ++k) scale = std::max(scale, norm(sub(P[(k + 1) % 4], P[k])));
        for (int k = 0; k < 4; ++k)
            if (std::fabs(dot(n, sub(P[(k + 1) % 4], P[k]))) > 1e-7 * nn * scale) return false;
        // strictly convex with one winding
        for (int k = 0; k < 4; ++k) {
            D3 e0 = sub(P[(k + 1) % 4], P[k]), e1 = sub(P[(k + 2) % 4], P[(k + 1) % 4]);
            if (dot(cross(e0, e1), n) <= 1e-9 * nn * norm(e0) * norm(e1)) return false;
        }
        q[0] = pa; q[1] = s0; q[2] = pb; q[3] = s1;
        return true;
    }
    return false;
}

inline uint64_t spread21(uint64_t v) {   // 21 bits -> every third bit
    v &= 0x1fffffULL;
    v = (v | v << 32) & 0x1f00000000ffffULL;
    v = (v | v << 16) & 0x1f0000ff0000ffULL;
    v = (v | v << 8) & 0x100f00f00f00f00fULL;
    v = (v | v << 4) & 0x10c30c30c30c30c3ULL;
    v = (v | v << 2) & 0x1249249249249249ULL;
    return v;
}

struct Item { uint64_t code; uint32_t id; };

void box_of_prim(const Prim& p, float lo[3], float hi[3]) {
    int nv = (p.flags & 1u) ? 4 : 3;
    for (int c = 0; c < 3; ++c) { lo[c] = p.v[c]; hi[c] = p.v[c]; }
    for (int k = 1; k < nv; ++k)
        for (int c = 0; c < 3; ++c) {
            lo[c] = std::min(lo[c], p.v[3 * k + c]);
            hi[c] = std::max(hi[c], p.v[3 * k + c]);
        }
}

// The uniform grid and the large-primitive leaves of one map (primitives mi.prim_begin .. mi.prim_end of h.prims).
void build_grid(HostHierarchy& h, MapInfo& mi) {
    const size_t p0 = mi.prim_begin, np = mi.prim_end - mi.prim_begin;
    std::vector<float> cx(np), cy(np), half(np);
    float x0 = 0.f, y0 = 0.f, x1 = 0.f, y1 = 0.f;
    for (size_t i = 0; i < np; ++i) {
        float lo[3], hi[3];
        box_of_prim(h.prims[p0 + i], lo, hi);
        cx[i] = 0.5f * (lo[0] + hi[0]); cy[i] = 0.5f * (lo[1] + hi[1]);
        // (rounded up a little: the margin derived from it must not fall short)
        half[i] = 0.5f * (float)std::sqrt((double)(hi[0] - lo[0]) * (hi[0] - lo[0]) + (double)(hi[1] - lo[1]) * (hi[1] - lo[1])) * 1.0001f + 1e-6f;
        if (i == 0 || cx[i] < x0) x0 = cx[i];
        if (i == 0 || cx[i] > x1) x1 = cx[i];
        if (i == 0 || cy[i] < y0) y0 = cy[i];
        if (i == 0 || cy[i] > y1) y1 = cy[i];
    }
    // cell size: about one primitive per cell, at most 1024 x 1024 cells
    const double ex = std::max((double)x1 - x0, 1e-3), ey = std::max((double)y1 - y0, 1e-3);
    double cell = std::sqrt(ex * ey / (double)std::max<size_t>(np, 1));
    cell = std::max(cell, std::max(ex, ey) / 1024.0);
    cell = std::max(cell, 1e-3);
    const uint32_t nx = (uint32_t)std::min(1024.0, std::floor(ex / cell) + 1.0), ny = (uint32_t)std::min(1024.0, std::floor(ey / cell) + 1.0);
    mi.gx0 = x0; mi.gy0 = y0; mi.cell = (float)cell; mi.inv_cell = (float)(1.0 / cell); mi.nx = nx; mi.ny = ny;
    mi.cell_begin = (uint32_t)h.cell_start.size();
    // small primitives by cell; the cell of a centre is computed exactly as the kernel computes the cells
    // of a range (same float32 expression), so a centre can never fall outside the range that covers it
    std::vector<uint32_t> cell_of(np, 0xffffffffu);
    std::vector<uint32_t> count((size_t)nx * ny + 1, 0u);
    float margin = 0.f;
    std::vector<Item> large;
    for (size_t i = 0; i < np; ++i) {
        if (half[i] <= 0.5f * mi.cell) {
            const float fx = std::floor((cx[i] - mi.gx0) * mi.inv_cell), fy = std::floor((cy[i] - mi.gy0) * mi.inv_cell);
            const uint32_t ix = (uint32_t)std::min((float)(nx - 1), std::max(0.f, fx)), iy = (uint32_t)std::min((float)(ny - 1), std::max(0.f, fy));
            cell_of[i] = iy * nx + ix;
            ++count[cell_of[i] + 1];
            margin = std::max(margin, half[i]);
        } else {
            uint64_t code = 0;
            const double ext = std::max(ex, ey);
            code |= spread21((uint64_t)std::min(2097151.0, std::max(0.0, (cx[i] - x0) / ext * 2097152.0)));
            code |= spread21((uint64_t)std::min(2097151.0, std::max(0.0, (cy[i] - y0) / ext * 2097152.0))) << 1;
            large.push_back({code, (uint32_t)i});
        }
    }
    // a float32 centre and the kernel's float32 range arithmetic differ by rounding: widen the margin
    mi.margin = margin * 1.0001f + 1e-4f * (1.f + std::fabs(x0) + std::fabs(y0) + (float)std::max(ex, ey));
    for (size_t c = 0; c < (size_t)nx * ny; ++c) count[c + 1] += count[c];
    const size_t base = h.grid_prims.size();
    h.grid_prims.resize(base + count[(size_t)nx * ny]);
    {
        std::vector<uint32_t> fill(count.begin(), count.end() - 1);
        for (size_t i = 0; i < np; ++i)
            if (cell_of[i] != 0xffffffffu) h.grid_prims[base + fill[cell_of[i]]++] = h.prims[p0 + i];
    }
    for (size_t c = 0; c <= (size_t)nx * ny; ++c) h.cell_start.push_back((uint32_t)(base + count[c]));
    // large primitives: Morton order, leaves of LARGE_LEAF_PRIMS
    std::sort(large.begin(), large.end(), [](const Item& a, const Item& b) { return a.code != b.code ? a.code < b.code : a.id < b.id; });
    mi.large_begin = (uint32_t)h.large_leaves.size();
    for (size_t i = 0; i < large.size(); i += LARGE_LEAF_PRIMS) {
        Node leaf;
        leaf.first = (uint32_t)h.grid_prims.size();
        leaf.count = (uint32_t)std::min<size_t>(LARGE_LEAF_PRIMS, large.size() - i);
        for (uint32_t k = 0; k < leaf.count; ++k) {
            float lo[3], hi[3];
            box_of_prim(h.prims[p0 + large[i + k].id], lo, hi);
            for (int c = 0; c < 3; ++c) {
                leaf.lo[c] = (k == 0) ? lo[c] : std::min(leaf.lo[c], lo[c]);
                leaf.hi[c] = (k == 0) ? hi[c] : std::max(leaf.hi[c], hi[c]);
            }
            h.grid_prims.push_back(h.prims[p0 + large[i + k].id]);
        }
        h.large_leaves.push_back(leaf);
    }
    mi.large_end = (uint32_t)h.large_leaves.size();
}

}  // namespace

HostHierarchy* build_hierarchy(int num_maps, const int64_t* tri_offset, const float* tri_xyz,
                               const uint8_t* tri_class, const float* tri_vis_cos, int agents_per_env, char* err, int err_len) {
    HostHierarchy* h = new HostHierarchy();
    h->maps.resize(num_maps);
    std::vector<Prim> local;
    std::vector<Item> items;
    for (int m = 0; m < num_maps; ++m) {
        int64_t t0 = tri_offset[m], t1 = tri_offset[m + 1];
        int64_t n = t1 - t0;
        if (n + 12LL * agents_per_env > (1LL << 24)) {
            std::snprintf(err, err_len, "map %d has %lld triangles; at most 2^24 - 12*A are supported", m, (long long)n);
            delete h;
            return nullptr;
        }
        // ---- primitives: fuse consecutive triangle pairs into quads where possible
        local.clear();
        for (int64_t i = 0; i < n;) {
            const F3* a = reinterpret_cast<const F3*>(tri_xyz + 9 * (t0 + i));
            Prim p;
            std::memset(&p, 0, sizeof(p));
            F3 q[4];
            bool quad = false;
            // (a triangle with a limited angular range is judged from its own centroid: never fused)
            const float vis = tri_vis_cos ? tri_vis_cos[t0 + i] : 0.f;
            const bool plain = !(vis > 0.f) && !(tri_vis_cos && i + 1 < n && tri_vis_cos[t0 + i + 1] > 0.f);
            if (plain && i + 1 < n && tri_class[t0 + i] == tri_class[t0 + i + 1]) {
                const F3* b = reinterpret_cast<const F3*>(tri_xyz + 9 * (t0 + i + 1));
                quad = fuse_quad(a, b, q);
            }
            if (!quad) { q[0] = a[0]; q[1] = a[1]; q[2] = a[2]; q[3] = a[2]; }
            for (int k = 0; k < 4; ++k) { p.v[3 * k] = q[k].x; p.v[3 * k + 1] = q[k].y; p.v[3 * k + 2] = q[k].z; }
            p.key_lo = ((0xFFFFFFu - (uint32_t)i) << 8) | tri_class[t0 + i];
            p.flags = quad ? 1u : 0u;
            p.vis_cos = vis > 0.f ? vis : 0.f;
            int nv = quad ? 4 : 3;
            for (int k = 0; k < nv; ++k)
                if (!lex_less(q[k], q[(k + 1) % nv])) p.flags |= 1u << (4 + k);
            local.push_back(p);
            i += quad ? 2 : 1;
        }
        // ---- classify long primitives, Morton-sort both classes
        size_t np = local.size();
        float mlo[3] = {0, 0, 0}, mhi[3] = {0, 0, 0};
        std::vector<float> diag(np);
        double mean_diag = 0.0;
        for (size_t i = 0; i < np; ++i) {
            float lo[3], hi[3];
            box_of_prim(local[i], lo, hi);
            for (int c = 0; c < 3; ++c) {
                if (i == 0 || lo[c] < mlo[c]) mlo[c] = lo[c];
                if (i == 0 || hi[c] > mhi[c]) mhi[c] = hi[c];
            }
            double dx = hi[0] - lo[0], dy = hi[1] - lo[1], dz = hi[2] - lo[2];
            diag[i] = (float)std::sqrt(dx * dx + dy * dy + dz * dz);
            mean_diag += diag[i];
        }
        if (np) mean_diag /= (double)np;
        double extent = std::max({(double)mhi[0] - mlo[0], (double)mhi[1] - mlo[1], (double)mhi[2] - mlo[2], 1e-30});
        items.clear();
        for (size_t i = 0; i < np; ++i) {
            float lo[3], hi[3];
            box_of_prim(local[i], lo, hi);
            uint64_t code = 0;
            for (int c = 0; c < 3; ++c) {
                double u = ((0.5 * ((double)lo[c] + hi[c])) - mlo[c]) / extent;
                uint64_t g = (uint64_t)std::min(2097151.0, std::max(0.0, u * 2097152.0));
                code |= spread21(g) << c;
            }
            bool is_long = diag[i] > 4.0 * mean_diag;
            items.push_back({code | (is_long ? (1ULL << 63) : 0ULL), (uint32_t)i});
        }
        std::sort(items.begin(), items.end(), [](const Item& a, const Item& b) {
            return a.code != b.code ? a.code < b.code : a.id < b.id;
        });
        // ---- leaves
        MapInfo& mi = h->maps[m];
        std::memset(&mi, 0, sizeof(mi));
        mi.n_tris = (uint32_t)n;
        mi.prim_begin = (uint32_t)h->prims.size();
        size_t leaf_begin = h->leaves.size();
        size_t i = 0;
        while (i < np) {
            bool is_long = (items[i].code >> 63) != 0;
            size_t cap = is_long ? LONG_LEAF_PRIMS : LEAF_PRIMS;
            size_t j = i;
            Node leaf;
            leaf.first = (uint32_t)h->prims.size();
            while (j < np && j - i < cap && ((items[j].code >> 63) != 0) == is_long) {
                const Prim& p = local[items[j].id];
                float lo[3], hi[3];
                box_of_prim(p, lo, hi);
                for (int c = 0; c < 3; ++c) {
                    leaf.lo[c] = (j == i) ? lo[c] : std::min(leaf.lo[c], lo[c]);
                    leaf.hi[c] = (j == i) ? hi[c] : std::max(leaf.hi[c], hi[c]);
                }
                h->prims.push_back(p);
                ++j;
            }
            leaf.count = (uint32_t)(j - i);
            h->leaves.push_back(leaf);
            i = j;
        }
        mi.prim_end = (uint32_t)h->prims.size();
        // ---- groups of consecutive leaves
        mi.group_begin = (uint32_t)h->groups.size();
        size_t leaf_end = h->leaves.size();
        for (size_t l = leaf_begin; l < leaf_end; l += GROUP_LEAVES) {
            Node g;
            g.first = (uint32_t)l;
            g.count = (uint32_t)std::min<size_t>(GROUP_LEAVES, leaf_end - l);
            for (uint32_t k = 0; k < g.count; ++k)
                for (int c = 0; c < 3; ++c) {
                    g.lo[c] = (k == 0) ? h->leaves[l + k].lo[c] : std::min(g.lo[c], h->leaves[l + k].lo[c]);
                    g.hi[c] = (k == 0) ? h->leaves[l + k].hi[c] : std::max(g.hi[c], h->leaves[l + k].hi[c]);
                }
            h->groups.push_back(g);
        }
        mi.group_end = (uint32_t)h->groups.size();
        build_grid(*h, mi);
        if (h->prims.size() >= (1ull << 28)) {
            std::snprintf(err, err_len, "more than 2^28 primitives in one scene");
            delete h;
            return nullptr;
        }
    }
    return h;
}

void free_hierarchy(HostHierarchy* h) { delete h; }
const Prim* hierarchy_prims(const HostHierarchy* h, size_t* n) { *n = h->prims.size(); return h->prims.data(); }
const Node* hierarchy_leaves(const HostHierarchy* h, size_t* n) { *n = h->leaves.size(); return h->leaves.data(); }
const Node* hierarchy_groups(const HostHierarchy* h, size_t* n) { *n = h->groups.size(); return h->groups.data(); }
const MapInfo* hierarchy_maps(const HostHierarchy* h, size_t* n) { *n = h->maps.size(); return h->maps.data(); }
const uint32_t* hierarchy_cell_start(const HostHierarchy* h, size_t* n) { *n = h->cell_start.size(); return h->cell_start.data(); }
const Prim* hierarchy_grid_prims(const HostHierarchy* h, size_t* n) { *n = h->grid_prims.size(); return h->grid_prims.data(); }
const Node* hierarchy_large_leaves(const HostHierarchy* h, size_t* n) { *n = h->large_leaves.size(); return h->large_leaves.data(); }

}  // namespace pic
