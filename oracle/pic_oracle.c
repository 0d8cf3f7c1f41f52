/*
 * pic_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, double-precision CPU statement of what the batched egocentric rasterizer
 * computes: for every requested (env, agent, camera) view and every pixel, a loop over ALL
 * primitives of the environment (every map triangle, then the 12 triangles of every other
 * active agent's box) -- no culling, no binning, no tiling.  It exists so that the CUDA path can
 * be compared against an independent definition; it shares no code with that path and nothing
 * in the product may call it (only tests, the smoke check and the benchmark's CPU-baseline leg).
 *
 * What is computed follows the paper's statement of the rasterizer (Sec. 3.2, Eq. 2: each
 * image is a deterministic function of the surrounding agents, the map geometry and one
 * camera of the ego-mounted rig; only the surroundings are drawn, never the ego itself) with the
 * frame conventions of its camera-rig table (agent frame x forward, y left, z up, yaw about z;
 * intrinsics given as a focal length in pixels, principal point at the image centre).  A rig row
 * is (mount x, y, z, yaw, pitch, fx, fy).  The paper fixes no
 * sampling, fill or depth rule; the ones used here are the steps O1..O12 below:
 *
 *  O1 camera      q = X - P_agent; q' = q - Rz(yaw_agent) m; X_c = (r.q', d.q', f.q') with
 *                 f = (cos(pitch)cos(a), cos(pitch)sin(a), sin(pitch)), r = (sin a, -cos a, 0), d = f x r,
 *                 a = yaw_agent + yaw_cam.  Pixel (u,v) samples the ray
 *                 rho = ((u+0.5-W/2)/fx, (v+0.5-H/2)/fy, 1).
 *  O2 background  world-z of the ray w = -rho_y cos(pitch) + sin(pitch); w<0 and camera above the
 *                 ground: class ground, depth min(far, C_z/(-w)); else sky at depth far.
 *  O3 primitives  map triangles in the given order (index 0..N-1), then box triangle t of agent b
 *                 at index N + 12 b + t (ego and inactive agents skipped).
 *  O4 coverage    N0=V1xV2, N1=V2xV0, N2=V0xV1, D=V0.N0 (sign-normalised to D>0), E_i = rho.N_i;
 *                 covered iff every E_i>0, or E_i==0 on a top-left edge (N_i.x>0, or ==0 and
 *                 N_i.y>0 -- fx, fy are positive so the division is dropped), and S=E0+E1+E2>0.
 *  O5 depth       z = D/S, kept iff near <= z <= far.
 *  O6 resolve     smallest z wins, exact ties go to the lower index; any kept fragment replaces
 *                 the background.
 *  O7 output      class u8, depth as f64 and rounded to binary16 (round-to-nearest-even).
 *  O8 ambiguity   pixels where a 1e-5 relative perturbation of an edge function, a depth gap, a
 *                 clip plane or the horizon could change the answer are flagged, so that a float32
 *                 implementation may legitimately differ there (and only there); so are pixels whose
 *                 winning primitive lies in a plane that passes the camera centre at less than 1/200
 *                 of its farthest vertex's distance (bit 16, informative): depth there is
 *                 ill-conditioned in float32 -- the per-pixel kappa output lets a comparison widen
 *                 its depth tolerance to 5e-7 * kappa, and depth gaps are judged with that width.
 *  O9 stepping    explicit-Euler kinematic bicycle update (pico_step).
 *  O10 road users and signals (Sec. 3.2, "Rendering features for driving": pedestrians, cyclists and
 *                 vehicles each in its own hue; traffic lights as disks visible only within a limited
 *                 angular range).  The paper gives neither formula, so the reading is: every agent may
 *                 carry its own class id (else the scene-wide one); a map triangle may carry a limit
 *                 c = cos(theta_max) > 0, and is then drawn in a view only if n.d >= c, where n is its
 *                 unit normal (V1-V0)x(V2-V0) by the order of its vertices and d the unit vector from
 *                 its centroid to the camera centre -- otherwise it is absent from that view, for all
 *                 pixels.  c = 0 (or no array) is the ordinary two-sided triangle.  A triangle within
 *                 1e-5 of its limit is drawn according to the exact comparison, and every pixel it
 *                 covers (or would cover) and could win is flagged (bit 32).
 *  O11 colour     (Sec. 3.2: the scene is drawn as flat-shaded primitives; agents are cuboids coloured per
 *                 face with depth-aware brightness, each kind of road user in its own hue.)  The paper gives
 *                 no numbers, so the reading is: a palette gives every class an 8-bit RGB triple; a map
 *                 triangle has its class's colour; face f of an agent's box has its class's colour times
 *                 s_f * beta(z), s = (rear 0.60, front 1.00, right 0.70, left 0.85, bottom 0.40, top 0.92),
 *                 beta(z) = 1 - 0.5 (z - near) / (far - near) with z the fragment's depth; ground and sky
 *                 have their classes' colours.  Without antialiasing a pixel shows the colour of its O6
 *                 winner (or of the background), rounded to 8 bits (floor(c + 0.5)).
 *  O12 antialiasing (Sec. 3.2: analytic-coverage antialiasing at a single sample per pixel, so that thin
 *                 structures stay visible at low resolution.)  No formula is given; the reading is a box
 *                 filter over the pixel's unit square, evaluated exactly:
 *                   - the edge functions E_i = rho.N_i and their sum S are linear in the pixel coordinates,
 *                     so the part of the pixel's square inside all three edges and within the depth range
 *                     (D/far <= S <= D/near) is a convex polygon; a primitive's coverage alpha is that
 *                     polygon's area (the square clipped by the five lines; for a single line crossing the
 *                     pixel this is the closed form of pico_edge_coverage);
 *                   - it leaves a fragment at every pixel with alpha > 0, at the depth z of its plane at the
 *                     pixel centre (the centre need not be covered), clamped to [near, far];
 *                   - the pixel's fragments are sorted by z (ties to the lower index) and composited front to
 *                     back, consecutive fragments of one surface -- map triangles of one class; the
 *                     triangles of one box -- first being merged into one layer: nearest first, each adds
 *                     its coverage (and its colour with that weight) until the layer's coverage A reaches 1:
 *                     C = sum_g T_g (sum_i a_i C_i) + T_end C_background, T_g = prod_{h<g} (1 - A_h);
 *                   - box triangles whose outer side is turned away from the camera centre are not drawn
 *                     (a box seen from outside looks the same without them, and they must not be merged
 *                     with the faces in front of them).
 *                 Pieces of one surface that tile the plane therefore add up to full coverage (no seams
 *                 inside a mesh, none along the edge between two faces of a box), and a strip thinner than a
 *                 pixel contributes its area.  Flags: 2 where two
 *                 fragments of different surfaces that both show are within the O8 depth width of each
 *                 other, or where a fragment covering less than 1e-3 of the pixel lies between two fragments of
 *                 one surface (whether those merge hangs on it), 8 on the horizon row
 *                 of a visible background, 32 as in O10.  Edge flags (1) do not apply: the colour is
 *                 continuous in the position of an edge.
 *
 * Parity pins: tests/test_oracle_*.py (closed forms, invariants, an independent ray caster,
 * hand-counted tiny scenes, numpy's binary16 conversion).  No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define REL_TOL 1e-5
#define GRAZING_KAPPA 200.0
#define DEPTH_KAPPA 5e-7      /* relative depth uncertainty of a float32 renderer per unit of kappa */

typedef struct { double x, y, z; } v3;

static v3 v3_sub(v3 a, v3 b) { v3 r = { a.x - b.x, a.y - b.y, a.z - b.z }; return r; }
static v3 v3_cross(v3 a, v3 b) {
    v3 r = { a.y * b.z - a.z * b.y, a.z * b.x - a.x * b.z, a.x * b.y - a.y * b.x };
    return r;
}
static double v3_dot(v3 a, v3 b) { return a.x * b.x + a.y * b.y + a.z * b.z; }
static double v3_norm(v3 a) { return sqrt(v3_dot(a, a)); }

/* One primitive of a view after O1/O4 set-up. */
typedef struct {
    v3 N[3];          /* sign-normalised edge normals */
    double D;         /* sign-normalised, > 0; 0 marks a skipped (degenerate / edge-on) primitive */
    double band[3];   /* O8 edge band without the |rho| factor */
    double kappa;     /* O8 (v): max|V_i| |N| / D, how close the primitive's plane passes by the camera centre */
    int32_t index;    /* global primitive index (O3) */
    uint8_t cls;
    uint8_t ghost;    /* O10: just outside its angular range -- not drawn, but its pixels are flagged */
    uint8_t unsure;   /* O10: within 1e-5 of its angular limit, on either side */
    uint8_t back;     /* O12: a box triangle whose outer side is turned away from the camera centre */
} prim_t;

typedef struct {
    v3 P;             /* agent position (z = 0) */
    v3 mw;            /* Rz(yaw_agent) * mount */
    v3 r, d, f;       /* camera basis in world coordinates */
    double fx, fy, cx, cy, pitch, cz;
} cam_t;

/* O1: world point -> camera space. */
static v3 to_camera(const cam_t* c, v3 X) {
    v3 q = v3_sub(X, c->P);
    v3 qp = v3_sub(q, c->mw);
    v3 r = { v3_dot(c->r, qp), v3_dot(c->d, qp), v3_dot(c->f, qp) };
    return r;
}

static void make_camera(cam_t* c, const float* pose, const float* cam, int H, int W) {
    double th = (double)pose[2];
    double mx = cam[0], my = cam[1], mz = cam[2], yaw = cam[3], pitch = cam[4];
    double a = th + yaw;
    c->P.x = pose[0]; c->P.y = pose[1]; c->P.z = 0.0;
    c->mw.x = cos(th) * mx - sin(th) * my;
    c->mw.y = sin(th) * mx + cos(th) * my;
    c->mw.z = mz;
    c->f.x = cos(pitch) * cos(a); c->f.y = cos(pitch) * sin(a); c->f.z = sin(pitch);
    c->r.x = sin(a); c->r.y = -cos(a); c->r.z = 0.0;
    c->d = v3_cross(c->f, c->r);
    c->fx = cam[5];                       /* focal lengths in pixels, as given */
    c->fy = cam[6];
    c->cx = W / 2.0; c->cy = H / 2.0;
    c->pitch = pitch;
    c->cz = mz;
}

/* O4 set-up of one triangle given in camera space. */
static void setup_prim(prim_t* p, v3 V0, v3 V1, v3 V2, int32_t index, uint8_t cls) {
    p->N[0] = v3_cross(V1, V2);
    p->N[1] = v3_cross(V2, V0);
    p->N[2] = v3_cross(V0, V1);
    p->D = v3_dot(V0, p->N[0]);
    if (p->D < 0.0) {
        for (int i = 0; i < 3; ++i) { p->N[i].x = -p->N[i].x; p->N[i].y = -p->N[i].y; p->N[i].z = -p->N[i].z; }
        p->D = -p->D;
    }
    /* edge i is opposite vertex i: (V1,V2), (V2,V0), (V0,V1) */
    double n0 = v3_norm(V0), n1 = v3_norm(V1), n2 = v3_norm(V2);
    p->band[0] = REL_TOL * fmax(n1, n2) * v3_norm(v3_sub(V2, V1));
    p->band[1] = REL_TOL * fmax(n2, n0) * v3_norm(v3_sub(V0, V2));
    p->band[2] = REL_TOL * fmax(n0, n1) * v3_norm(v3_sub(V1, V0));
    {
        v3 Nn = v3_cross(v3_sub(V1, V0), v3_sub(V2, V0));
        p->kappa = (p->D > 0.0) ? fmax(n0, fmax(n1, n2)) * v3_norm(Nn) / p->D : 0.0;
    }
    p->index = index;
    p->cls = cls;
    p->ghost = 0;
    p->unsure = 0;
    p->back = 0;
}

/* O10: cosine of the angle between the triangle's normal (by vertex order) and the direction from its
   centroid to the camera centre (the origin of camera space). */
static double facing_cosine(v3 V0, v3 V1, v3 V2) {
    v3 nrm = v3_cross(v3_sub(V1, V0), v3_sub(V2, V0));
    v3 g = { (V0.x + V1.x + V2.x) / 3.0, (V0.y + V1.y + V2.y) / 3.0, (V0.z + V1.z + V2.z) / 3.0 };
    double nn = v3_norm(nrm), gn = v3_norm(g);
    if (nn == 0.0 || gn == 0.0) return -2.0;        /* degenerate, or the camera sits on the centroid: never in range */
    return -v3_dot(nrm, g) / (nn * gn);
}

/* O3: the 12 triangles of agent b's box, in world coordinates. */
static void box_triangles(const float* pose, const float* dim, v3 tri[12][3]) {
    static const int face[6][4] = {
        {0, 2, 6, 4},  /* rear  (-x) */
        {1, 5, 7, 3},  /* front (+x) */
        {0, 4, 5, 1},  /* right (-y) */
        {2, 3, 7, 6},  /* left  (+y) */
        {0, 1, 3, 2},  /* bottom     */
        {4, 6, 7, 5},  /* top        */
    };
    double x = pose[0], y = pose[1], th = pose[2];
    double hl = dim[0] / 2.0, hw = dim[1] / 2.0, h = dim[2];
    v3 c[8];
    for (int i = 0; i < 8; ++i) {
        double sx = (i & 1) ? hl : -hl;
        double sy = (i & 2) ? hw : -hw;
        c[i].x = x + cos(th) * sx - sin(th) * sy;
        c[i].y = y + sin(th) * sx + cos(th) * sy;
        c[i].z = (i & 4) ? h : 0.0;
    }
    for (int f = 0; f < 6; ++f) {
        tri[2 * f][0] = c[face[f][0]]; tri[2 * f][1] = c[face[f][1]]; tri[2 * f][2] = c[face[f][2]];
        tri[2 * f + 1][0] = c[face[f][0]]; tri[2 * f + 1][1] = c[face[f][2]]; tri[2 * f + 1][2] = c[face[f][3]];
    }
}

/* O7: double -> IEEE binary16 bits, round-to-nearest-even (default rounding mode assumed). */
uint16_t pico_f64_to_f16(double z) {
    uint16_t sign = 0;
    if (z != z) return 0x7e00;
    if (z < 0.0) { sign = 0x8000; z = -z; }
    if (z == 0.0) return sign;
    if (isinf(z)) return sign | 0x7c00;
    int e;
    (void)frexp(z, &e);               /* z = m 2^e, 0.5 <= m < 1  => exponent of the leading bit is e-1 */
    int lead = e - 1;
    if (lead < -14) lead = -14;       /* subnormal quantum 2^-24 */
    double quantum = ldexp(1.0, lead - 10);
    double r = nearbyint(z / quantum);   /* exact scaling, ties-to-even */
    if (r >= 2048.0) { r /= 2.0; lead += 1; }
    if (lead > 15) return sign | 0x7c00;
    if (r < 1024.0) return sign | (uint16_t)r;     /* subnormal (lead == -14) */
    return sign | (uint16_t)(((lead + 15) << 10) | ((int)r - 1024));
}

/* Sutherland-Hodgman clip of a convex polygon against a.x*X + a.y*Y + a.z*Z + w >= 0. */
static int clip_poly(const v3* in, int n, v3 a, double w, v3* out) {
    int m = 0;
    for (int i = 0; i < n; ++i) {
        v3 p = in[i], q = in[(i + 1) % n];
        double dp = v3_dot(a, p) + w, dq = v3_dot(a, q) + w;
        if (dp >= 0.0) out[m++] = p;
        if ((dp >= 0.0) != (dq >= 0.0)) {
            double t = dp / (dp - dq);
            v3 x = { p.x + t * (q.x - p.x), p.y + t * (q.y - p.y), p.z + t * (q.z - p.z) };
            out[m++] = x;
        }
    }
    return m;
}

/* Does the camera-space triangle meet the view frustum (closed)?  Only used for the work counts. */
static int meets_frustum(v3 V0, v3 V1, v3 V2, double tx, double ty, double near, double far) {
    v3 a[16], b[16];
    a[0] = V0; a[1] = V1; a[2] = V2;
    int n = 3;
    v3 pl[6] = { {0, 0, 1}, {0, 0, -1}, {1, 0, tx}, {-1, 0, tx}, {0, 1, ty}, {0, -1, ty} };
    double w[6] = { -near, far, 0, 0, 0, 0 };
    for (int i = 0; i < 6 && n > 0; ++i) {
        n = clip_poly(a, n, pl[i], w[i], b);
        memcpy(a, b, sizeof(v3) * (size_t)n);
    }
    return n > 0;
}

/* O3 + O4: every primitive of environment e as seen by camera c of ego a (the ego and inactive agents are
   skipped), in index order; *t_vis counts those that meet the frustum (work counts only).  NULL on
   allocation failure; the caller frees. */
static prim_t* view_prims(const cam_t* c, int e, int a, int A, int H, int W, double near, double far,
                          const int32_t* env_map_id, const int64_t* map_tri_offset,
                          const float* tri_xyz, const uint8_t* tri_class, int agent_class,
                          const float* poses, const float* dims, const uint8_t* active,
                          const uint8_t* agent_classes, const float* tri_vis_cos,
                          int64_t* np_out, int64_t* n_map_out, int64_t* t_vis_out)
{
    int m = env_map_id[e];
    int64_t t0 = map_tri_offset[m], t1 = map_tri_offset[m + 1];
    int64_t n_map = t1 - t0;
    int64_t n_prim = n_map + 12 * (int64_t)A;
    prim_t* prim = (prim_t*)malloc(sizeof(prim_t) * (size_t)(n_prim > 0 ? n_prim : 1));
    if (!prim) return NULL;
    int64_t np = 0, t_vis = 0;
    double tx = (W / 2.0) / c->fx, ty = (H / 2.0) / c->fy;
    for (int64_t t = 0; t < n_map; ++t) {
        const float* p = tri_xyz + 9 * (size_t)(t0 + t);
        v3 X0 = { p[0], p[1], p[2] }, X1 = { p[3], p[4], p[5] }, X2 = { p[6], p[7], p[8] };
        v3 V0 = to_camera(c, X0), V1 = to_camera(c, X1), V2 = to_camera(c, X2);
        setup_prim(&prim[np], V0, V1, V2, (int32_t)t, tri_class[t0 + t]);
        if (tri_vis_cos && tri_vis_cos[t0 + t] > 0.0f) {          /* O10: one-sided, limited angular range */
            double lim = (double)tri_vis_cos[t0 + t], cosang = facing_cosine(V0, V1, V2);
            if (fabs(cosang - lim) <= REL_TOL) prim[np].unsure = 1;
            if (!(cosang >= lim)) {
                if (prim[np].unsure) prim[np].ghost = 1;
                else prim[np].D = 0.0;                             /* absent from this view */
            }
        }
        if (prim[np].D != 0.0 && !prim[np].ghost && meets_frustum(V0, V1, V2, tx, ty, near, far)) ++t_vis;
        ++np;
    }
    for (int b = 0; b < A; ++b) {
        if (b == a) continue;                                   /* the ego is never drawn */
        if (active && !active[(size_t)e * A + b]) continue;
        v3 tri[12][3];
        box_triangles(poses + 3 * ((size_t)e * A + b), dims + 3 * ((size_t)e * A + b), tri);
        v3 centre = { poses[3 * ((size_t)e * A + b)], poses[3 * ((size_t)e * A + b) + 1], 0.5 * dims[3 * ((size_t)e * A + b) + 2] };
        v3 Bc = to_camera(c, centre);
        for (int t = 0; t < 12; ++t) {
            v3 V0 = to_camera(c, tri[t][0]), V1 = to_camera(c, tri[t][1]), V2 = to_camera(c, tri[t][2]);
            setup_prim(&prim[np], V0, V1, V2, (int32_t)(n_map + 12 * b + t),
                       agent_classes ? agent_classes[(size_t)e * A + b] : (uint8_t)agent_class);
            {   /* O12: the camera centre (the origin) and the box's centre on the same side of the triangle's plane */
                v3 nrm = v3_cross(v3_sub(V1, V0), v3_sub(V2, V0));
                double s_cam = -v3_dot(nrm, V0), s_box = v3_dot(nrm, v3_sub(Bc, V0));
                prim[np].back = !(s_cam * s_box < 0.0);
            }
            if (prim[np].D != 0.0 && meets_frustum(V0, V1, V2, tx, ty, near, far)) ++t_vis;
            ++np;
        }
    }
    *np_out = np; *n_map_out = n_map; *t_vis_out = t_vis;
    return prim;
}

/*
 * Render the listed views.  view_ids[i] = (e*A + a)*K + k.  Outputs are [n_views, H, W]:
 *   out_class  u8      O6/O7 class
 *   out_depth  f64     O5/O6 depth (metres along the optical axis)
 *   out_f16    u16     O7 binary16 bits of the depth
 *   out_index  i32     global index of the winning primitive, -1 for background
 *   out_flag   u8      O8 bit mask: 1 edge, 2 depth gap, 4 near/far plane, 8 horizon, 16 grazing plane (informative),
 *                      32 a triangle at the limit of its angular range (O10)
 *   agent_classes u8 [E,A] or NULL (every agent has class agent_class); tri_vis_cos f32 [N] or NULL (O10)
 *   out_kappa  f64     conditioning of the winner's depth: max|V_i| |N| / D of its plane (0 for background);
 *                      a float32 renderer's depth may be off by about 5e-7 * kappa relative
 *   counts     i64 [n_views,4]: primitives meeting the frustum, primitives with >=1 kept
 *              fragment, kept fragments, flagged pixels
 * Any output pointer may be NULL.  Returns 0, or -1 on allocation failure.
 */
int pico_render(int E, int A, int K, int H, int W, double near, double far,
                const int32_t* env_map_id, const int64_t* map_tri_offset,
                const float* tri_xyz, const uint8_t* tri_class,
                int agent_class, int sky_class, int ground_class,
                const float* poses, const float* dims, const uint8_t* active, const float* rig,
                const uint8_t* agent_classes, const float* tri_vis_cos,
                int n_views, const int64_t* view_ids,
                uint8_t* out_class, double* out_depth, uint16_t* out_f16, int32_t* out_index,
                uint8_t* out_flag, double* out_kappa, int64_t* counts, int n_threads)
{
    (void)E;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#else
    (void)n_threads;
#endif
    int failed = 0;
    for (int vi = 0; vi < n_views; ++vi) {
        int64_t id = view_ids[vi];
        int k = (int)(id % K);
        int a = (int)((id / K) % A);
        int e = (int)(id / ((int64_t)K * A));
        size_t base = (size_t)vi * (size_t)H * (size_t)W;
        const float* cam = rig + 7 * k;

        /* inactive ego: sky everywhere */
        if (active && !active[(size_t)e * A + a]) {
            for (size_t p = 0; p < (size_t)H * W; ++p) {
                if (out_class) out_class[base + p] = (uint8_t)sky_class;
                if (out_depth) out_depth[base + p] = far;
                if (out_f16) out_f16[base + p] = pico_f64_to_f16(far);
                if (out_index) out_index[base + p] = -1;
                if (out_flag) out_flag[base + p] = 0;
                if (out_kappa) out_kappa[base + p] = 0.0;
            }
            if (counts) memset(counts + 4 * (size_t)vi, 0, 4 * sizeof(int64_t));
            continue;
        }

        cam_t c;
        make_camera(&c, poses + 3 * ((size_t)e * A + a), cam, H, W);

        /* O3 + O4 set-up of every primitive of the environment */
        int64_t np = 0, n_map = 0, t_vis = 0;
        prim_t* prim = view_prims(&c, e, a, A, H, W, near, far, env_map_id, map_tri_offset, tri_xyz, tri_class, agent_class,
                                  poses, dims, active, agent_classes, tri_vis_cos, &np, &n_map, &t_vis);
        uint8_t* hit = prim ? (uint8_t*)calloc((size_t)np + 1, 1) : NULL;
        if (!prim || !hit) { free(prim); free(hit); failed = 1; break; }

        int64_t n_frag = 0, n_flag = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : n_frag, n_flag)
        for (int v = 0; v < H; ++v) {
            for (int u = 0; u < W; ++u) {
                v3 rho = { (u + 0.5 - c.cx) / c.fx, (v + 0.5 - c.cy) / c.fy, 1.0 };
                double rho_n = v3_norm(rho);

                /* O4-O6: nearest kept fragment */
                double z_win = 0.0, k_win = 0.0; int32_t i_win = -1; uint8_t c_win = 0;
                for (int64_t j = 0; j < np; ++j) {
                    const prim_t* p = &prim[j];
                    if (p->D == 0.0 || p->ghost) continue;
                    int covered = 1;
                    double S = 0.0;
                    for (int i = 0; i < 3; ++i) {
                        double Ei = v3_dot(rho, p->N[i]);
                        S += Ei;
                        if (Ei > 0.0) continue;
                        if (Ei == 0.0 && (p->N[i].x > 0.0 || (p->N[i].x == 0.0 && p->N[i].y > 0.0))) continue;
                        covered = 0;
                    }
                    if (!covered || !(S > 0.0)) continue;
                    double z = p->D / S;
                    if (z < near || z > far) continue;
                    ++n_frag;
                    if (!hit[j]) {
#pragma omp atomic write
                        hit[j] = 1;
                    }
                    if (i_win < 0 || z < z_win || (z == z_win && p->index < i_win)) {
                        z_win = z; i_win = p->index; c_win = p->cls; k_win = p->kappa;
                    }
                }

                /* O2: background */
                double w = -rho.y * cos(c.pitch) + sin(c.pitch);
                uint8_t cls; double depth;
                if (i_win >= 0) { cls = c_win; depth = z_win; }
                else if (w < 0.0 && c.cz > 0.0) { cls = (uint8_t)ground_class; depth = fmin(far, c.cz / (-w)); }
                else { cls = (uint8_t)sky_class; depth = far; }

                /* O8: ambiguity mask */
                uint8_t flag = 0;
                if (i_win < 0 && fabs(w) <= REL_TOL) flag |= 8;
                /* (v) the winner's plane grazes the camera centre: a 6e-8 relative change of its
                   camera-space vertices (float32 spacing) moves the depth by more than half the
                   1e-4 tolerance */
                if (i_win >= 0 && k_win > GRAZING_KAPPA) flag |= 16;
                for (int64_t j = 0; j < np; ++j) {
                    const prim_t* p = &prim[j];
                    if (p->D == 0.0) continue;
                    double Ei[3], S = 0.0;
                    int inside_band = 1, on_band = 0, covered = 1;
                    for (int i = 0; i < 3; ++i) {
                        Ei[i] = v3_dot(rho, p->N[i]);
                        S += Ei[i];
                        double band = p->band[i] * rho_n;
                        if (Ei[i] < -band) inside_band = 0;
                        if (fabs(Ei[i]) <= band) on_band = 1;
                        if (!(Ei[i] > 0.0 ||
                              (Ei[i] == 0.0 && (p->N[i].x > 0.0 || (p->N[i].x == 0.0 && p->N[i].y > 0.0)))))
                            covered = 0;
                    }
                    if (!(S > 0.0)) continue;
                    double z = p->D / S;
                    int could_show = (i_win < 0) || (z <= (1.0 + REL_TOL) * z_win);
                    /* (i) pixel centre within the band of p's boundary */
                    if (inside_band && on_band && could_show &&
                        z >= near * (1.0 - REL_TOL) && z <= far * (1.0 + REL_TOL)) flag |= 1;
                    if (!covered) continue;
                    /* (vi) O10: a triangle at the limit of its angular range that covers the pixel and could win */
                    if (p->unsure && z >= near && z <= far && could_show) flag |= 32;
                    if (p->ghost) continue;
                    /* (ii) a kept fragment of another class almost as near as the winner */
                    if (i_win >= 0 && z >= near && z <= far && p->cls != c_win &&
                        fabs(z - z_win) <= fmax(REL_TOL, DEPTH_KAPPA * fmax(p->kappa, k_win)) * z_win) flag |= 2;
                    /* (iii) a covered fragment sitting on the near or far plane that matters */
                    if ((fabs(z - near) <= REL_TOL * near || fabs(z - far) <= REL_TOL * far) && could_show) flag |= 4;
                }
                if (flag) ++n_flag;

                size_t o = base + (size_t)v * W + u;
                if (out_class) out_class[o] = cls;
                if (out_depth) out_depth[o] = depth;
                if (out_f16) out_f16[o] = pico_f64_to_f16(depth);
                if (out_index) out_index[o] = i_win;
                if (out_flag) out_flag[o] = flag;
                if (out_kappa) out_kappa[o] = (i_win >= 0) ? k_win : 0.0;
            }
        }
        if (counts) {
            int64_t t_hit = 0;
            for (int64_t j = 0; j < np; ++j) t_hit += hit[j];
            counts[4 * (size_t)vi + 0] = t_vis;
            counts[4 * (size_t)vi + 1] = t_hit;
            counts[4 * (size_t)vi + 2] = n_frag;
            counts[4 * (size_t)vi + 3] = n_flag;
        }
        free(prim);
        free(hit);
    }
    return failed ? -1 : 0;
}

/* O12, one edge alone (kept for the pins of the clipper below, which the renderer uses): fraction of the unit
   square around a pixel centre on which a linear function is positive, given its
   value e0 at the centre and its increments a, b per pixel in x and y.  With A = |a|, B = |b| the function
   ranges over e0 +- (A + B)/2 on the square; the fraction is 1/2 + e0/max(A,B) on the middle stretch
   |e0| <= |A - B|/2 (the boundary crosses two opposite sides) and a quadratic where it cuts off a corner. */
double pico_edge_coverage(double e0, double a, double b) {
    double A = fabs(a), B = fabs(b);
    double h = 0.5 * (A + B);
    if (e0 >= h) return (e0 > 0.0 || h > 0.0) ? 1.0 : 0.0;     /* (a constant zero function is nowhere positive) */
    if (e0 <= -h) return 0.0;
    double hi = fmax(A, B), lo = fmin(A, B), g = 0.5 * (hi - lo);
    if (fabs(e0) <= g) return 0.5 + e0 / hi;
    if (e0 < 0.0) return (e0 + h) * (e0 + h) / (2.0 * A * B);
    return 1.0 - (h - e0) * (h - e0) / (2.0 * A * B);
}

/* O12: area of the part of the unit square around a pixel centre on which all nl (at most 8) linear functions
   e[i] + a[i] x + b[i] y are non-negative (Sutherland-Hodgman clipping of the square, then the shoelace formula). */
double pico_pixel_coverage(int nl, const double* e, const double* a, const double* b) {
    double px[16] = { -0.5, 0.5, 0.5, -0.5 }, py[16] = { -0.5, -0.5, 0.5, 0.5 };
    int n = 4;
    for (int i = 0; i < nl && n > 0; ++i) {
        double qx[16], qy[16];
        int m = 0;
        for (int k = 0; k < n; ++k) {
            int k1 = (k + 1) % n;
            double f0 = e[i] + a[i] * px[k] + b[i] * py[k], f1 = e[i] + a[i] * px[k1] + b[i] * py[k1];
            if (f0 >= 0.0) { qx[m] = px[k]; qy[m] = py[k]; ++m; }
            if ((f0 >= 0.0) != (f1 >= 0.0)) {
                double t = f0 / (f0 - f1);
                qx[m] = px[k] + t * (px[k1] - px[k]); qy[m] = py[k] + t * (py[k1] - py[k]); ++m;
            }
        }
        n = m;
        memcpy(px, qx, sizeof(double) * (size_t)n);
        memcpy(py, qy, sizeof(double) * (size_t)n);
    }
    if (n < 3) return 0.0;
    double twice = 0.0;
    for (int k = 0; k < n; ++k) { int k1 = (k + 1) % n; twice += px[k] * py[k1] - px[k1] * py[k]; }
    return 0.5 * fabs(twice);
}

static const double FACE_SHADE[6] = { 0.60, 1.00, 0.70, 0.85, 0.40, 0.92 };   /* rear, front, right, left, bottom, top */

/* O11: colour (0..255 per channel, not yet rounded) of a fragment of primitive p at depth z. */
static void shade(const prim_t* p, int64_t n_map, double z, double near, double far, const uint8_t* palette, double rgb[3]) {
    double k = 1.0;
    if (p->index >= n_map) {
        int face = (int)((p->index - n_map) % 12) / 2;
        k = FACE_SHADE[face] * (1.0 - 0.5 * (z - near) / (far - near));
    }
    for (int ch = 0; ch < 3; ++ch) rgb[ch] = k * (double)palette[3 * p->cls + ch];
}

/* O12: which fragments merge -- map triangles of one class; the triangles of one box. */
static int64_t surface_of(const prim_t* p, int64_t n_map) {
    return (p->index < n_map) ? (int64_t)p->cls : 256 + (p->index - n_map) / 12;
}
/* (ii) of O8 in colour: do two primitives show different colours -- another class, or another face of a box */
static int64_t colour_of(const prim_t* p, int64_t n_map) {
    return (p->index < n_map) ? (int64_t)p->cls : 256 + (p->index - n_map) / 2;
}

typedef struct { double z, alpha, kappa; int64_t j; } frag_t;

static int frag_before(const frag_t* a, const frag_t* b, const prim_t* prim) {
    return a->z < b->z || (a->z == b->z && prim[a->j].index < prim[b->j].index);
}

/*
 * Render the listed views in colour (O11), optionally antialiased (O12).  Arguments as pico_render;
 *   palette  u8 [256,3]  RGB of every class
 *   aa       0: a pixel shows its O6 winner; 1: analytic coverage (O12)
 *   out_rgb  u8  [n_views,H,W,3]   rounded colour
 *   out_rgbf f64 [n_views,H,W,3]   the colour before rounding (0..255)
 *   out_flag u8  [n_views,H,W]     aa 0: the O8 mask of pico_render with "another class" read as "another
 *                                  surface or class" in (ii); aa 1: the flags listed under O12
 * Any output pointer may be NULL.  Returns 0, or -1 on allocation failure.
 */
int pico_render_rgb(int E, int A, int K, int H, int W, double near, double far,
                    const int32_t* env_map_id, const int64_t* map_tri_offset,
                    const float* tri_xyz, const uint8_t* tri_class,
                    int agent_class, int sky_class, int ground_class,
                    const float* poses, const float* dims, const uint8_t* active, const float* rig,
                    const uint8_t* agent_classes, const float* tri_vis_cos,
                    const uint8_t* palette, int aa,
                    int n_views, const int64_t* view_ids,
                    uint8_t* out_rgb, double* out_rgbf, uint8_t* out_flag, int n_threads)
{
    (void)E;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#else
    (void)n_threads;
#endif
    int failed = 0;
    for (int vi = 0; vi < n_views; ++vi) {
        int64_t id = view_ids[vi];
        int k = (int)(id % K);
        int a = (int)((id / K) % A);
        int e = (int)(id / ((int64_t)K * A));
        size_t base = (size_t)vi * (size_t)H * (size_t)W;
        const float* cam = rig + 7 * k;
        if (active && !active[(size_t)e * A + a]) {          /* inactive ego: sky everywhere */
            for (size_t p = 0; p < (size_t)H * W; ++p) {
                for (int ch = 0; ch < 3; ++ch) {
                    if (out_rgb) out_rgb[3 * (base + p) + ch] = palette[3 * sky_class + ch];
                    if (out_rgbf) out_rgbf[3 * (base + p) + ch] = (double)palette[3 * sky_class + ch];
                }
                if (out_flag) out_flag[base + p] = 0;
            }
            continue;
        }
        cam_t c;
        make_camera(&c, poses + 3 * ((size_t)e * A + a), cam, H, W);
        int64_t np = 0, n_map = 0, t_vis = 0;
        prim_t* prim = view_prims(&c, e, a, A, H, W, near, far, env_map_id, map_tri_offset, tri_xyz, tri_class, agent_class,
                                  poses, dims, active, agent_classes, tri_vis_cos, &np, &n_map, &t_vis);
        if (!prim) { failed = 1; break; }
        int alloc_failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
        for (int v = 0; v < H; ++v) {
            frag_t* fr = aa ? (frag_t*)malloc(sizeof(frag_t) * (size_t)(np > 0 ? np : 1)) : NULL;
            if (aa && !fr) {
#pragma omp atomic write
                alloc_failed = 1;
                continue;
            }
            for (int u = 0; u < W; ++u) {
                v3 rho = { (u + 0.5 - c.cx) / c.fx, (v + 0.5 - c.cy) / c.fy, 1.0 };
                double rho_n = v3_norm(rho);
                double w = -rho.y * cos(c.pitch) + sin(c.pitch);
                int bg_ground = (w < 0.0 && c.cz > 0.0);
                int bg_class = bg_ground ? ground_class : sky_class;
                double rgb[3] = { 0.0, 0.0, 0.0 };
                uint8_t flag = 0;
                if (!aa) {
                    /* O4-O6 as in pico_render */
                    double z_win = 0.0, k_win = 0.0; int64_t j_win = -1;
                    for (int64_t j = 0; j < np; ++j) {
                        const prim_t* p = &prim[j];
                        if (p->D == 0.0 || p->ghost) continue;
                        int covered = 1;
                        double S = 0.0;
                        for (int i = 0; i < 3; ++i) {
                            double Ei = v3_dot(rho, p->N[i]);
                            S += Ei;
                            if (Ei > 0.0) continue;
                            if (Ei == 0.0 && (p->N[i].x > 0.0 || (p->N[i].x == 0.0 && p->N[i].y > 0.0))) continue;
                            covered = 0;
                        }
                        if (!covered || !(S > 0.0)) continue;
                        double z = p->D / S;
                        if (z < near || z > far) continue;
                        if (j_win < 0 || z < z_win || (z == z_win && p->index < prim[j_win].index)) { z_win = z; j_win = j; k_win = p->kappa; }
                    }
                    if (j_win >= 0) shade(&prim[j_win], n_map, z_win, near, far, palette, rgb);
                    else for (int ch = 0; ch < 3; ++ch) rgb[ch] = (double)palette[3 * bg_class + ch];
                    /* O8 with surfaces in place of classes in (ii) */
                    if (j_win < 0 && fabs(w) <= REL_TOL) flag |= 8;
                    if (j_win >= 0 && k_win > GRAZING_KAPPA) flag |= 16;
                    for (int64_t j = 0; j < np; ++j) {
                        const prim_t* p = &prim[j];
                        if (p->D == 0.0) continue;
                        double S = 0.0;
                        int inside_band = 1, on_band = 0, covered = 1;
                        for (int i = 0; i < 3; ++i) {
                            double Ei = v3_dot(rho, p->N[i]);
                            S += Ei;
                            double band = p->band[i] * rho_n;
                            if (Ei < -band) inside_band = 0;
                            if (fabs(Ei) <= band) on_band = 1;
                            if (!(Ei > 0.0 || (Ei == 0.0 && (p->N[i].x > 0.0 || (p->N[i].x == 0.0 && p->N[i].y > 0.0))))) covered = 0;
                        }
                        if (!(S > 0.0)) continue;
                        double z = p->D / S;
                        int could_show = (j_win < 0) || (z <= (1.0 + REL_TOL) * z_win);
                        if (inside_band && on_band && could_show && z >= near * (1.0 - REL_TOL) && z <= far * (1.0 + REL_TOL)) flag |= 1;
                        if (!covered) continue;
                        if (p->unsure && z >= near && z <= far && could_show) flag |= 32;
                        if (p->ghost) continue;
                        if (j_win >= 0 && z >= near && z <= far &&
                            (p->cls != prim[j_win].cls || colour_of(p, n_map) != colour_of(&prim[j_win], n_map)) &&
                            fabs(z - z_win) <= fmax(REL_TOL, DEPTH_KAPPA * fmax(p->kappa, k_win)) * z_win) flag |= 2;
                        if ((fabs(z - near) <= REL_TOL * near || fabs(z - far) <= REL_TOL * far) && could_show) flag |= 4;
                    }
                } else {
                    /* O12: the pixel's fragments */
                    int64_t nf = 0;
                    int unsure = 0;
                    for (int64_t j = 0; j < np; ++j) {
                        const prim_t* p = &prim[j];
                        if (p->D == 0.0 || p->back) continue;
                        double S = 0.0, Ei[5], ax[5], by[5];
                        ax[3] = 0.0; by[3] = 0.0;
                        for (int i = 0; i < 3; ++i) {
                            Ei[i] = v3_dot(rho, p->N[i]);
                            ax[i] = p->N[i].x / c.fx;                /* increments of E_i per pixel in x and y */
                            by[i] = p->N[i].y / c.fy;
                            S += Ei[i];
                            ax[3] += ax[i]; by[3] += by[i];
                        }
                        Ei[3] = S - p->D / far;  /* z <= far */
                        Ei[4] = p->D / near - S; ax[4] = -ax[3]; by[4] = -by[3];   /* z >= near */
                        double alpha = pico_pixel_coverage(5, Ei, ax, by);
                        if (!(alpha > 0.0)) continue;
                        double z = (S > 0.0) ? p->D / S : far;
                        if (z < near) z = near;
                        if (z > far) z = far;
                        if (p->unsure && alpha >= 1e-3) unsure = 1;
                        if (p->ghost) continue;
                        fr[nf].z = z; fr[nf].alpha = alpha; fr[nf].kappa = p->kappa; fr[nf].j = j;
                        ++nf;
                    }
                    for (int64_t i = 1; i < nf; ++i) {          /* insertion sort by (z, index) */
                        frag_t x = fr[i];
                        int64_t q = i;
                        while (q > 0 && frag_before(&x, &fr[q - 1], prim)) { fr[q] = fr[q - 1]; --q; }
                        fr[q] = x;
                    }
                    /* front to back, the fragments of one surface merged into one layer */
                    double T = 1.0;
                    int64_t shown_end = 0;                      /* fragments [0, shown_end) show */
                    for (int64_t i = 0; i < nf && T > 0.0;) {
                        int64_t surf = surface_of(&prim[fr[i].j], n_map);
                        double Acc = 0.0, sum[3] = { 0.0, 0.0, 0.0 };
                        int64_t q = i;
                        while (q < nf && surface_of(&prim[fr[q].j], n_map) == surf) {
                            /* nearer fragments first: each adds its coverage until the layer is full */
                            double col[3], add = fmin(fr[q].alpha, 1.0 - Acc);
                            shade(&prim[fr[q].j], n_map, fr[q].z, near, far, palette, col);
                            for (int ch = 0; ch < 3; ++ch) sum[ch] += add * col[ch];
                            Acc += add;
                            ++q;
                        }
                        for (int ch = 0; ch < 3; ++ch) rgb[ch] += T * sum[ch];
                        T *= 1.0 - Acc;
                        i = q;
                        shown_end = q;
                    }
                    for (int ch = 0; ch < 3; ++ch) rgb[ch] += T * (double)palette[3 * bg_class + ch];
                    /* flags */
                    if (T > 1e-3 && fabs(w) <= REL_TOL) flag |= 8;
                    if (unsure) flag |= 32;
                    /* a fragment of negligible coverage (below 1e-3: a renderer in float32 may not see it at all) that
                       separates two fragments of one surface decides whether those merge: ambiguous */
                    for (int64_t i = 0; i < nf && i <= shown_end; ++i) {
                        if (fr[i].alpha >= 1e-3) continue;
                        int64_t q = i + 1;
                        while (q < nf && fr[q].alpha < 1e-3) ++q;
                        if (i >= 1 && q < nf && surface_of(&prim[fr[i - 1].j], n_map) == surface_of(&prim[fr[q].j], n_map) &&
                            surface_of(&prim[fr[i].j], n_map) != surface_of(&prim[fr[q].j], n_map)) flag |= 2;
                    }
                    for (int64_t i = 0; i + 1 < shown_end + 1 && i + 1 < nf; ++i) {
                        /* neighbours in depth order of different surfaces, the nearer of which shows */
                        const frag_t *x = &fr[i], *y = &fr[i + 1];
                        if (i >= shown_end) break;
                        if (surface_of(&prim[x->j], n_map) == surface_of(&prim[y->j], n_map)) continue;
                        if (x->alpha < 1e-3 && y->alpha < 1e-3) continue;
                        if (fabs(y->z - x->z) <= fmax(REL_TOL, DEPTH_KAPPA * fmax(x->kappa, y->kappa)) * x->z) flag |= 2;
                    }
                }
                size_t o = base + (size_t)v * W + u;
                for (int ch = 0; ch < 3; ++ch) {
                    if (out_rgbf) out_rgbf[3 * o + ch] = rgb[ch];
                    if (out_rgb) out_rgb[3 * o + ch] = (uint8_t)floor(rgb[ch] + 0.5);
                }
                if (out_flag) out_flag[o] = flag;
            }
            free(fr);
        }
        free(prim);
        if (alloc_failed) { failed = 1; break; }
    }
    return failed ? -1 : 0;
}

/*
 * O9: one explicit-Euler step of the kinematic bicycle model, everything from the old state:
 *   x' = x + v cos(yaw) dt,  y' = y + v sin(yaw) dt,  yaw' = yaw + (v / wheelbase) tan(steer) dt,
 *   v' = clamp(v + accel dt, 0, v_max).   state f64 [n,4] (x, y, yaw, v) in place;
 *   actions f32 [n,2] (accel, steer); inactive agents do not move.
 */
void pico_step(double* state, const float* actions, const uint8_t* active, int64_t n,
               double dt, double wheelbase, double v_max)
{
    for (int64_t i = 0; i < n; ++i) {
        if (active && !active[i]) continue;
        double x = state[4 * i], y = state[4 * i + 1], th = state[4 * i + 2], v = state[4 * i + 3];
        double acc = actions[2 * i], steer = actions[2 * i + 1];
        state[4 * i + 0] = x + v * cos(th) * dt;
        state[4 * i + 1] = y + v * sin(th) * dt;
        state[4 * i + 2] = th + (v / wheelbase) * tan(steer) * dt;
        double vn = v + acc * dt;
        if (vn < 0.0) vn = 0.0;
        if (vn > v_max) vn = v_max;
        state[4 * i + 3] = vn;
    }
}

int pico_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
