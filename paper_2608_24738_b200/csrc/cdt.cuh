// Taxicab / chessboard distance transform and the brute-force distance transform (paper, Section 2.3.2).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace tmcdt {

constexpr int kBig = 1 << 29;  // "no background seen yet"; adding an extent to it does not overflow

struct PassParams {
    const uint8_t* mask;   // first pass: the input mask
    const int32_t* in;     // later passes
    int32_t* out;
    int64_t total;         // voxels of the batch
    int64_t inner;         // view (outer, n, inner)
    int n;
    int first, last;       // first pass reads the mask; last pass turns "no background" into -1
};

// One axis: g_new(x) = min_j op(g(x with x_k := j), |x_k - j|), op = + (taxicab) or max (chessboard).  A thread owns
// one voxel and scans outward; every candidate at distance d is worth at least d, so the scan stops once d reaches
// the minimum found so far.  Consecutive threads are consecutive in memory for every axis.
template <bool CHESS>
__global__ void __launch_bounds__(256) cdt_axis_kernel(const __grid_constant__ PassParams P) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= P.total) return;
    const int y = (int)((e / P.inner) % P.n);
    auto value = [&](int64_t idx) -> int { return P.first ? (P.mask[idx] != 0 ? kBig : 0) : P.in[idx]; };
    int best = value(e);
    const int up = y, dn = P.n - 1 - y;
    for (int d = 1; d < best && (d <= up || d <= dn); ++d) {
        if (d <= up) { const int v = value(e - (int64_t)d * P.inner); best = min(best, CHESS ? max(v, d) : v + d); }
        if (d <= dn) { const int v = value(e + (int64_t)d * P.inner); best = min(best, CHESS ? max(v, d) : v + d); }
    }
    P.out[e] = (P.last && best >= kBig) ? -1 : best;
}

// ---- brute force ----
struct BruteParams {
    const uint8_t* mask;
    const int32_t* sites;    // (images, V): linear indices of the background voxels of each image, in any order
    const int32_t* counts;   // (images)
    float* out;
    int V;
    int ext[4];
    float w[4];
};

// Background voxels of every image -> its list (order does not matter: the minimum is taken over all of them).
__global__ void __launch_bounds__(256) collect_background_kernel(const uint8_t* mask, int32_t* sites, int32_t* counts,
                                                                 int64_t total, int V) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= total) return;
    if (mask[e] == 0) {
        const int64_t img = e / V;
        const int slot = atomicAdd(counts + img, 1);
        sites[img * V + slot] = (int)(e - img * V);
    }
}

template <int RANK>
__device__ __forceinline__ void split(int lin, const int* ext, int* x) {
#pragma unroll
    for (int a = RANK - 1; a >= 0; --a) { x[a] = lin % ext[a]; lin /= ext[a]; }
}

// Every voxel against every background voxel of its image; the block's image is blockIdx.y.
template <int METRIC, int RANK>
__global__ void __launch_bounds__(256) brute_kernel(const __grid_constant__ BruteParams P) {
    __shared__ int s_x[RANK][256];
    const int img = blockIdx.y;
    const int vox = blockIdx.x * blockDim.x + threadIdx.x;
    const bool act = vox < P.V;
    int x[RANK];
    split<RANK>(act ? vox : 0, P.ext, x);
    const int count = P.counts[img];
    float best = __int_as_float(0x7f800000);
    for (int t0 = 0; t0 < count; t0 += 256) {
        __syncthreads();
        if (t0 + threadIdx.x < count) {
            int sx[RANK];
            split<RANK>(P.sites[(int64_t)img * P.V + t0 + threadIdx.x], P.ext, sx);
#pragma unroll
            for (int a = 0; a < RANK; ++a) s_x[a][threadIdx.x] = sx[a];
        }
        __syncthreads();
        const int m = min(256, count - t0);
        for (int s = 0; s < m; ++s) {
            float d = 0.f;
#pragma unroll
            for (int a = 0; a < RANK; ++a) {
                const float t = P.w[a] * fabsf((float)(x[a] - s_x[a][s]));
                d = METRIC == 0 ? fmaf(t, t, d) : (METRIC == 1 ? d + t : fmaxf(d, t));
            }
            best = fminf(best, d);
        }
    }
    if (act) P.out[(int64_t)img * P.V + vox] = METRIC == 0 ? sqrtf(best) : best;
}

}  // namespace tmcdt
