// Device/host data layout of the rasterizer library (internal).
#pragma once
#include <stdint.h>
#include <vector_types.h>

namespace pic {

constexpr int TILE = 64;        // a view is rendered in tiles of up to TILE x TILE pixels (one CTA each)
constexpr int MAX_CAMS = 16;    // cameras per rig
constexpr int LEAF_PRIMS = 8;   // primitives per leaf (8 threads per leaf in the cull pass)
constexpr int LONG_LEAF_PRIMS = 8;   // long primitives get leaves of their own so the others' boxes stay tight
constexpr int GROUP_LEAVES = 32;     // leaves per group (one per lane)
constexpr int LARGE_LEAF_PRIMS = 4;  // primitives per leaf of the large-primitive list

// Map primitive in hierarchy order: a triangle, or a planar convex quad fused from two consecutive
// triangles of the input that share an edge (same class).  64 bytes, read as four 128-bit loads.
struct Prim {
    float v[12];        // 4 vertices xyz in perimeter order (triangle: the 4th repeats the 3rd)
    uint32_t key_lo;    // (0xFFFFFF - primitive index) << 8 | class : low half of the z-buffer key
    uint32_t flags;     // bit 0: quad; bits 4..7: edge i runs against its canonical direction
    float vis_cos;      // > 0: drawn only from its front side and within acos(vis_cos) of its normal (triangles only)
    uint32_t pad;
};
static_assert(sizeof(Prim) == 64, "Prim must be 64 bytes");

// Axis-aligned box of a leaf (over primitives) or a group (over leaves); 32 bytes.
struct Node {
    float lo[3];
    uint32_t first;
    float hi[3];
    uint32_t count;
};
static_assert(sizeof(Node) == 32, "Node must be 32 bytes");

struct MapInfo {
    uint32_t group_begin, group_end;   // range in the groups array
    uint32_t n_tris;                   // triangles of the map as given (box indices start here)
    uint32_t prim_begin;               // first primitive (used by the exhaustive kernel)
    uint32_t prim_end;
    // uniform grid over the map's ground-plane extent (the cull kernel's structure, see pic_bvh.cpp)
    uint32_t cell_begin;               // first entry of this map in the cell-start array (nx * ny + 1 entries)
    uint32_t nx, ny;                   // cells per row, rows
    float gx0, gy0;                    // corner of cell (0, 0)
    float cell, inv_cell;              // cell size, its reciprocal
    float margin;                      // no small primitive reaches farther than this from the centre of its box (xy)
    uint32_t large_begin, large_end;   // range in the large-primitive leaves
    uint32_t pad;
};
static_assert(sizeof(MapInfo) == 64, "MapInfo must be 64 bytes");

// Per-agent geometry written once per render by the agent kernel; 32 bytes.
struct AgentGeom {
    float x, y;       // box centre on the ground plane
    float c, s;       // cos, sin of the heading
    float hl, hw, h;  // half length, half width, height
    uint32_t active;  // 0: inactive; else 1 | class of the agent's box << 8
};

struct CamConst {
    float mx, my, mz;
    float cpsi, spsi, cphi, sphi;   // cos/sin of the camera yaw and pitch (rounded from double)
    float fx, fy;
};

// Per-view camera written by the agent kernel: ego position, mount and rotation rows; 64 bytes.
struct ViewCam {
    float px, py;              // ego position
    float mwx, mwy, mwz;       // mount in world axes
    float rx, ry;              // right   (rz = 0)
    float dx, dy, dz;          // down
    float fx, fy, fz;          // forward
    float pad[3];
};
static_assert(sizeof(ViewCam) == 64, "ViewCam must be 64 bytes");

// Per-camera tables shared by all views of a call: ray coordinates of pixel columns / rows and the
// background (analytic ground plane / sky) of every row.
struct RigTables {
    const float* ray_x;        // [K][W]
    const float* ray_y;        // [K][H]
    const float* bg_z;         // [K][H] background depth
    const uint32_t* bg_cls;    // [K][H] background class
};

struct RenderParams {
    int32_t E, A, K, H, W;
    int32_t tiles_x, tiles_y;
    float near_z, far_z;
    float w_near, w_far;            // 1/near, 1/far: kept range of the reciprocal depth
    uint32_t cls_agent, cls_sky, cls_ground;
    const int32_t* env_map;
    const MapInfo* env_maps;        // [E] the MapInfo of each environment's map (one load instead of two)
    const MapInfo* maps;
    const Node* groups;
    const Node* leaves;
    const Prim* prims;
    const uint32_t* cell_start;     // grid: per map nx * ny + 1 offsets into grid_prims
    const Prim* grid_prims;         // the primitives in grid order: small ones cell by cell (row-major), then the large ones leaf by leaf
    const Node* large_leaves;       // boxes over up to LARGE_LEAF_PRIMS consecutive large primitives of grid_prims
    const AgentGeom* agents;
    const ViewCam* cams;            // [E*A*K]
    RigTables rig;
    uint8_t* out_class;
    uint16_t* out_depth;
    float* out_depth32;             // optional
    unsigned long long* counters;   // optional [16]
    uint32_t* occlusion;            // optional [E*A*K][A][2]: per view and other agent, visible pixels and pixels its box covers alone
    uint8_t* out_rgb;               // colour output [E*A*K][H][W][3] (colour kernel only)
    const uint8_t* palette;         // [256][3] RGB of every class (colour kernel only)
    uint32_t* status;               // the scene's sticky status word
    uint32_t* overflow;             // [1 + tiles of all views]: count, then the tiles left to the cooperative kernel
    uint2* surv;                    // per tile: the cull kernel's survivors (head + list), read by the render kernel
    int32_t debug_flags;            // bit 0: no per-cell trivial accept/reject, bit 1: record pool / list of 2 entries, bit 2: cooperative kernel only, bit 3: pool of 40, bits 4-7: profiling stop
    uint32_t n_jobs;                // tiles to render in this launch (views x tiles per view); set by the launcher
    long long view_first;           // render views [view_first, view_first + gridDim / tiles)
    CamConst cam[MAX_CAMS];
};

// Host-side result of the hierarchy build for all maps of a scene.
struct HostHierarchy;
HostHierarchy* build_hierarchy(int num_maps, const int64_t* tri_offset, const float* tri_xyz,
                               const uint8_t* tri_class, const float* tri_vis_cos, int agents_per_env, char* err, int err_len);
void free_hierarchy(HostHierarchy*);
const Prim* hierarchy_prims(const HostHierarchy*, size_t* n);
const Node* hierarchy_leaves(const HostHierarchy*, size_t* n);
const Node* hierarchy_groups(const HostHierarchy*, size_t* n);
const MapInfo* hierarchy_maps(const HostHierarchy*, size_t* n);
const uint32_t* hierarchy_cell_start(const HostHierarchy*, size_t* n);
const Prim* hierarchy_grid_prims(const HostHierarchy*, size_t* n);
const Node* hierarchy_large_leaves(const HostHierarchy*, size_t* n);

}  // namespace pic
