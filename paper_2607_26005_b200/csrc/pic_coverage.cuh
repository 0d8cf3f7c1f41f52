// Analytic coverage of a pixel (internal; included by pic_colour.cuh): the area of the pixel's unit square on the
// inner side of one line (closed form) or of six lines (a record's four edges and the two lines at which its
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

// Area of the part of the unit square around a pixel centre on which all six e[i] + a[i] x + b[i] y >= 0 (a
// record's four edges and the two lines at which its plane reaches the far and the near depth).
// The region is convex; its area is half the sum over its boundary lines -- the square's four sides and the
// six lines -- of (distance of the line from the centre) x (length of the line's piece on the boundary); the
// piece is found by cutting the line with all other constraints.  Written with t measured along (B, -A), which
// keeps the interior on the left: the contribution of line j is C_j (t1 - t0).  Two lines that (nearly)
// coincide and face the same way -- an edge along a side of the pixel -- must not both claim the same piece:
// constraint m is moved by 1e-5 pixel, inwards when it cuts such a line of higher index and outwards otherwise,
// so exactly one of the two keeps the piece whatever the rounding.  (Two coinciding lines that face each
// other bound a sliver; both keep their piece and the two contributions cancel.)
constexpr int CLINES = 6;
__device__ __forceinline__ float pixel_coverage(const float (&e)[CLINES], const float (&a)[CLINES], const float (&b)[CLINES]) {
    constexpr int N = 4 + CLINES;
    float A[N], B[N], C[N], nudge[N];
    A[0] = 1.f; A[1] = -1.f; A[2] = 0.f; A[3] = 0.f;
    B[0] = 0.f; B[1] = 0.f; B[2] = 1.f; B[3] = -1.f;
#pragma unroll
    for (int m = 0; m < 4; ++m) C[m] = 0.5f;
#pragma unroll
    for (int m = 0; m < CLINES; ++m) { A[4 + m] = a[m]; B[4 + m] = b[m]; C[4 + m] = e[m]; }
#pragma unroll
    for (int m = 0; m < N; ++m) nudge[m] = 1e-5f * (fabsf(A[m]) + fabsf(B[m]));
    float twice = 0.f;
#pragma unroll
    for (int j = 0; j < N; ++j) {
        const float n2 = fm(A[j], A[j], mul(B[j], B[j]));
        if (n2 > 0.f) {
            const float k = -__fdividef(C[j], n2), p0x = k * A[j], p0y = k * B[j];     // the line's point nearest the centre
            float t0 = -3e38f, t1 = 3e38f;
#pragma unroll
            for (int m = 0; m < N; ++m) {
                if (m == j) continue;
                const float be = fm(A[m], B[j], -mul(B[m], A[j]));
                const bool same_side = m < j && fm(A[m], A[j], mul(B[m], B[j])) > 0.f;
                const float al = fm(A[m], p0x, fm(B[m], p0y, C[m])) + (same_side ? -nudge[m] : nudge[m]);
                const float t = -__fdividef(al, be);
                if (be > 0.f) t0 = fmaxf(t0, t);
                else if (be < 0.f) t1 = fminf(t1, t);
                else if (al < 0.f) t1 = -3e38f;                                          // parallel and outside
            }
            if (t1 > t0) twice = fm(C[j], t1 - t0, twice);
        }
    }
    return fminf(fmaxf(0.5f * twice, 0.f), 1.f);
}

}  // namespace pic
