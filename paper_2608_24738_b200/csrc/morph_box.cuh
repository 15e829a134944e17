// Flat box elements on float32 images (paper, Section 2.3.1: erosion / dilation with a flat structuring element are
// a minimum / maximum over the footprint).  The minimum over a box is the minimum over its rows of the minima along
// the rows, and every border rule acts on one axis at a time, so a box of odd extents centred on its voxel is run as
// passes of one kernel, box_strip_kernel: a window of +-RH positions along the contiguous axis combined with a window
// of +-RV positions along one other axis (the "walk" axis).  The first pass takes the last two axes together, every
// earlier axis is a pass with RH = 0.  A lane owns four consecutive voxels of a row (16-byte loads and stores) and a
// strip of T positions of the walk axis: it loads the T + 2 RV rows its strip needs once, all loads in flight
// together, reduces every row along the contiguous axis (neighbouring quads by warp shuffle) and then combines
// 2 RV + 1 reduced rows per output row from registers.  Both border rules are applied in the kernel: rows beyond the
// walk axis are mapped (or take the constant) as whole rows, and only the first and the last lane of a warp fetch
// positions beside their quad from memory, through the border rule at the ends of a row.
// Requires a contiguous extent that is a multiple of 4 and 16-byte aligned buffers.
#pragma once
#include <cuda_runtime.h>
#include <limits.h>
#include <stdint.h>

#include "morph.cuh"

namespace tmmorph {

struct StripParams {
    const float* in;
    float* out;
    int W;                // contiguous extent (voxels per row)
    int n;                // extent of the walk axis
    int inner;            // rows per position of the walk axis (walk_stride / W)
    int64_t walk_stride;  // voxels between consecutive positions of the walk axis
    unsigned chunks;      // 128-voxel chunks per row
    unsigned strip_groups;// groups of 8 strips per column of the walk axis
    int mode;             // border rule of both axes
    float cval;           // value of the constant rule
    int reverse;          // walk the blocks backwards (every second pass: it starts with what the pass before wrote last)
};

template <bool MIN> __device__ __forceinline__ float pick(float a, float b) { return MIN ? fminf(a, b) : fmaxf(a, b); }

// Folds the positions left (l: x0 - R .. x0 - 1) and right (r: x0 + 4 .. x0 + 3 + R) of a quad into the window
// minima of its four voxels: voxel j reaches l[k] for k >= j and r[k] for k <= j + R - 4.
template <bool MIN, int R>
__device__ __forceinline__ void box_fold_sides(float (&h)[4], const float (&l)[R > 0 ? R : 1], const float (&r)[R > 0 ? R : 1]) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int k = 0; k < R; ++k) {
            if (k >= j) h[j] = pick<MIN>(h[j], l[k]);
            if (k <= j + R - 4) h[j] = pick<MIN>(h[j], r[k]);
        }
    }
}

// The strip of one lane.  ROWS_IN: every row of the strip and of its halo lies inside the walk axis (no border rule
// along it); x_in: every window position of the warp lies inside the row.
template <bool MIN, int RH, int RV, int T, bool ROWS_IN>
__device__ __forceinline__ void box_strip_body(const StripParams& P, const int64_t base, const int p0, const int x0,
                                               const bool act, const bool first, const bool last, const bool x_in) {
    constexpr int ROWS = T + 2 * RV;
    constexpr int RQ = RH > 0 ? RH : 1;
    const float neutral = MIN ? __int_as_float(0x7f800000) : __int_as_float(0xff800000);
    // every row of the strip and its halo, all loads in flight together; pm: the row after the border rule, -1 for
    // a row of the constant
    float h[ROWS][4];
    int pm[ROWS];
#pragma unroll
    for (int k = 0; k < ROWS; ++k) {
        int p = p0 - RV + k;
        pm[k] = ROWS_IN || map_coord(p, P.n, P.mode) ? p : -1;
        float4 c = make_float4(P.cval, P.cval, P.cval, P.cval);
        if ((ROWS_IN || pm[k] >= 0) && act) c = *reinterpret_cast<const float4*>(P.in + base + (int64_t)pm[k] * P.walk_stride);
        h[k][0] = c.x; h[k][1] = c.y; h[k][2] = c.z; h[k][3] = c.w;
    }
    if (RH > 0) {
        // along the row: the quad's own positions, then those of the neighbouring lanes
#pragma unroll
        for (int k = 0; k < ROWS; ++k) {
            float l[RQ], r[RQ];
#pragma unroll
            for (int q = 0; q < RH; ++q) {
                l[q] = __shfl_up_sync(0xffffffffu, h[k][4 - RH + q], 1);
                r[q] = __shfl_down_sync(0xffffffffu, h[k][q], 1);
                if (first) l[q] = neutral;  // fetched below
                if (last) r[q] = neutral;
            }
            float v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                v[j] = h[k][j];
#pragma unroll
                for (int d = -RH; d <= RH; ++d)
                    if (d != 0 && j + d >= 0 && j + d < 4) v[j] = pick<MIN>(v[j], h[k][j + d]);
            }
            box_fold_sides<MIN, RH>(v, l, r);
#pragma unroll
            for (int j = 0; j < 4; ++j) h[k][j] = v[j];
        }
        if (act && (first || last)) {
            // positions no neighbouring lane holds, one side per lane (the first lane its left, the last lane its right;
            // a lane that is both takes the right side in a second round): offsets against x0 after the border rule,
            // INT_MIN for the constant
#pragma unroll 1
            for (int round = 0; round < 2; ++round) {
                const bool left = first && round == 0;
                int off[RQ];
#pragma unroll
                for (int q = 0; q < RH; ++q) {
                    int c = left ? x0 - RH + q : x0 + 4 + q;
                    off[q] = x_in || map_coord(c, P.W, P.mode) ? c - x0 : INT_MIN;
                }
#pragma unroll
                for (int k = 0; k < ROWS; ++k) {
                    const float* row = P.in + base + (int64_t)pm[k] * P.walk_stride;
                    float l[RQ], r[RQ];
#pragma unroll
                    for (int q = 0; q < RH; ++q) {
                        const float e = (ROWS_IN || pm[k] >= 0) && off[q] != INT_MIN ? row[off[q]] : P.cval;
                        l[q] = left ? e : neutral;
                        r[q] = left ? neutral : e;
                    }
                    box_fold_sides<MIN, RH>(h[k], l, r);
                }
                if (!(first && last)) break;
            }
        }
    }
    if (!act) return;
#pragma unroll
    for (int t = 0; t < T; ++t) {
        if (!ROWS_IN && p0 + t >= P.n) break;
        float4 a = make_float4(h[t][0], h[t][1], h[t][2], h[t][3]);
#pragma unroll
        for (int k = 1; k <= 2 * RV; ++k) {
            a.x = pick<MIN>(a.x, h[t + k][0]); a.y = pick<MIN>(a.y, h[t + k][1]);
            a.z = pick<MIN>(a.z, h[t + k][2]); a.w = pick<MIN>(a.w, h[t + k][3]);
        }
        *reinterpret_cast<float4*>(P.out + base + (int64_t)(p0 + t) * P.walk_stride) = a;
    }
}

// Block = 8 strips x 32 quads.  Blocks enumerate (column of the walk axis, group of 8 strips, chunk of 128 voxels),
// chunk fastest.  A column is a pair (index over the axes before the walk axis, row within one position of it).
template <bool MIN, int RH, int RV, int T>
__global__ void __launch_bounds__(256, (RH <= 1 && RV <= 1) ? 3 : 2) box_strip_kernel(const __grid_constant__ StripParams P) {
    unsigned b = P.reverse ? gridDim.x - 1 - blockIdx.x : blockIdx.x;
    const unsigned ch = b % P.chunks; b /= P.chunks;
    const unsigned sg = b % P.strip_groups;
    const unsigned col = b / P.strip_groups;
    const int p0 = (int)(sg * 8 + threadIdx.y) * T;  // first position of the strip
    if (p0 >= P.n) return;                           // the whole warp leaves
    const int lane = threadIdx.x;
    const int x0 = (int)(ch * 32 + lane) * 4;
    const bool act = x0 < P.W;                       // lanes beyond the row stay for the shuffles
    const bool first = lane == 0, last = lane == 31 || x0 + 4 >= P.W;
    const bool x_in = (int)ch * 128 - RH >= 0 && (int)ch * 128 + 128 + RH <= P.W;
    const unsigned o = col / (unsigned)P.inner, i = col - o * (unsigned)P.inner;
    const int64_t base = (int64_t)o * P.n * P.walk_stride + (int64_t)i * P.W + (act ? x0 : 0);
    if (p0 - RV >= 0 && p0 + T + RV <= P.n) box_strip_body<MIN, RH, RV, T, true>(P, base, p0, x0, act, first, last, x_in);
    else box_strip_body<MIN, RH, RV, T, false>(P, base, p0, x0, act, first, last, x_in);
}

// Positions of the walk axis per strip for a window of +-RV: the strip and its halo stay within 12 rows of registers.
__host__ __device__ constexpr int box_strip_len(int RV) { return RV <= 2 ? 8 : 4; }

}  // namespace tmmorph
