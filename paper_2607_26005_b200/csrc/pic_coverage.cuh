// Analytic coverage of a pixel (internal; included by pic_colour.cuh): the area of the pixel's unit square on the
// inner side of one line (closed form) or of several lines (a record's four edges and the two lines at which its
// plane reaches the far and the near depth).
#pragma once
#include "pic_device.cuh"

namespace pic {

// Fraction of the unit square around a pixel centre on which e0 + a x + b y > 0 (one line crossing the pixel).
__device__ __forceinline__ float edge_coverage(float e0, float a, float b) {
    const float A = fabsf(a), B = fabsf(b), h = 0.5f * (A + B);
    if (e0 >= h) return 1.f;
    if (e0 <= -h) return 0.f;
    const float hi = fmaxf(A, B), lo = fminf(A, B), g = 0.5f * (hi - lo);
    if (fabsf(e0) <= g) return 0.5f + __fdividef(e0, hi);
    const float d = h - fabsf(e0), corner = __fdividef(d * d, 2.f * A * B);     // the corner triangle cut off
    return e0 < 0.f ? corner : 1.f - corner;
}

// Area of the part of the unit square around a pixel centre on which all NL lines e[i] + a[i] x + b[i] y >= 0 (of a
// record's four edges and the two lines at which its plane reaches the far and the near depth, all six or those
// that cross the pixel; an unused slot holds the constant 1).
// The region is convex; its area is half the sum over its boundary lines -- the square's four sides and the
// six lines -- of (distance of the line from the centre) x (length of the line's piece on the boundary); the
// piece is found by cutting the line with all other constraints.  Written with t measured along (B, -A), which
// keeps the interior on the left: the contribution of line j is C_j (t1 - t0).  Two lines that (nearly)
// coincide and face the same way -- an edge along a side of the pixel -- must not both claim the same piece:
// constraint m is moved by 1e-5 pixel, inwards when it cuts such a line of higher index and outwards otherwise,
// so exactly one of the two keeps the piece whatever the rounding.  (Two coinciding lines that face each
// other bound a sliver; both keep their piece and the two contributions cancel.)
constexpr int CLINES = 6;
template <int NL>
__device__ __forceinline__ float pixel_coverage(const float (&e)[NL], const float (&a)[NL], const float (&b)[NL]) {
    constexpr int N = 4 + NL;
    float A[N], B[N], C[N];
    A[0] = 1.f; A[1] = -1.f; A[2] = 0.f; A[3] = 0.f;
    B[0] = 0.f; B[1] = 0.f; B[2] = 1.f; B[3] = -1.f;
#pragma unroll
    for (int m = 0; m < 4; ++m) C[m] = 0.5f;
#pragma unroll
    for (int m = 0; m < NL; ++m) { A[4 + m] = a[m]; B[4 + m] = b[m]; C[4 + m] = e[m]; }
    float twice = 0.f;
    // A loop over the boundary lines that is NOT unrolled (the code stays small enough for the instruction cache):
    // the line in turn sits in slot 0 and the arrays are rotated by one slot per turn, so slot p holds line
    // (j + p) mod N, which has a lower index than line j exactly when p >= N - j.
#pragma unroll 1
    for (int j = 0; j < N; ++j) {
        const float n2 = fm(A[0], A[0], mul(B[0], B[0]));
        const float k = -__fdividef(C[0], n2), p0x = k * A[0], p0y = k * B[0];     // the line's point nearest the centre
        float t0 = -3e38f, t1 = 3e38f;
#pragma unroll
        for (int p = 1; p < N; ++p) {
            const float be = fm(A[p], B[0], -mul(B[p], A[0]));
            const bool same_side = p >= N - j && fm(A[p], A[0], mul(B[p], B[0])) > 0.f;
            const float nudge = 1e-5f * (fabsf(A[p]) + fabsf(B[p]));
            const float al = fm(A[p], p0x, fm(B[p], p0y, C[p])) + (same_side ? -nudge : nudge);
            const float t = -__fdividef(al, be);
            // (written with selects: the lanes of a warp rarely agree on the sign of be)
            t0 = be > 0.f ? fmaxf(t0, t) : t0;
            t1 = be < 0.f ? fminf(t1, t) : t1;
            t1 = (be == 0.f && al < 0.f) ? -3e38f : t1;                                  // parallel and outside
        }
        // (a constant, n2 == 0 -- a triangle's fourth edge, an unused slot -- bounds nothing)
        twice = (n2 > 0.f && t1 > t0) ? fm(C[0], t1 - t0, twice) : twice;
        const float ra = A[0], rb = B[0], rc = C[0];
#pragma unroll
        for (int p = 0; p + 1 < N; ++p) { A[p] = A[p + 1]; B[p] = B[p + 1]; C[p] = C[p + 1]; }
        A[N - 1] = ra; B[N - 1] = rb; C[N - 1] = rc;
    }
    return fminf(fmaxf(0.5f * twice, 0.f), 1.f);
}

}  // namespace pic
