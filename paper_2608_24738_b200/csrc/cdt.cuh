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

// First axis (contiguous lines of up to 8192 voxels): one warp per line, lanes take consecutive voxels.  The zero
// bits of the line are collected as ballot words in shared memory; a voxel finds its nearest zero to the left and
// to the right inside its own word with __clz / __ffs and otherwise takes the last zero before / first zero
// after the word.  The 1-D distance is the same for both metrics.
struct RowParams {
    const uint8_t* mask;
    int32_t* out;
    int64_t rows;
    int n0;
    int last;
};

__global__ void __launch_bounds__(256) cdt_row_kernel(const __grid_constant__ RowParams P) {
    constexpr int MAXW = 256;
    __shared__ uint32_t s_word[8][MAXW];
    __shared__ int s_next[8][MAXW];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + warp;
    if (row >= P.rows) return;  // the whole warp leaves together
    const int n0 = P.n0, W = (n0 + 31) >> 5;
    const uint8_t* src = P.mask + row * n0;
    bool any = false;
    for (int b = 0; b < W; ++b) {
        const int x = 32 * b + lane;
        const unsigned word = __ballot_sync(0xffffffffu, x < n0 && src[x] == 0);
        if (lane == 0) s_word[warp][b] = word;
        any = any || word != 0u;
    }
    __syncwarp();
    if (lane == 0) {
        int nxt = 1 << 20;
        for (int b = W - 1; b >= 0; --b) {
            s_next[warp][b] = nxt;
            const uint32_t word = s_word[warp][b];
            if (word) nxt = 32 * b + __ffs(word) - 1;
        }
    }
    __syncwarp();
    int carry = -(1 << 20);  // last zero before word b
    for (int b = 0; b < W; ++b) {
        const uint32_t word = s_word[warp][b];
        const int x = 32 * b + lane;
        const uint32_t ml = word & (0xffffffffu >> (31 - lane)), mr = word >> lane;
        const int zl = ml ? 32 * b + 31 - __clz(ml) : carry;
        const int zr = mr ? x + __ffs(mr) - 1 : s_next[warp][b];
        if (x < n0) P.out[row * n0 + x] = any ? min(x - zl, zr - x) : (P.last ? -1 : kBig);
        if (word) carry = 32 * b + 31 - __clz(word);
    }
}

// A further axis of up to 1024 rows: a block stages an (n x CW) strip of values in shared memory (rows of 128 or
// 64 contiguous bytes) and a warp scans four consecutive rows of its 32 columns at a time, so that every row fetched
// from the tile serves four voxels.  The nearest candidate of a step is d rows away, which ends the scan once d
// reaches the largest of the four minima.
// CW: columns of a strip (32, or 16 for long axes: half the shared memory per block, two row groups per warp).
template <bool CHESS, int CW>
__global__ void __launch_bounds__(512) cdt_strip_kernel(const __grid_constant__ PassParams P, const int strips_per_slab) {
    extern __shared__ __align__(16) int sm_cdt[];  // [n][CW]
    const int n = P.n;
    const int64_t slab = blockIdx.x / strips_per_slab;
    const int64_t c0 = (int64_t)(blockIdx.x - slab * strips_per_slab) * CW;
    const int64_t base = slab * (int64_t)n * P.inner + c0;
    const int width = (int)min((int64_t)CW, P.inner - c0);
    constexpr int TPR = CW / 4;
    if ((P.inner & 3) == 0) {  // rows are 16-byte aligned: CW / 4 threads copy one row
#pragma unroll 4
        for (int t = threadIdx.x; t < n * TPR; t += blockDim.x) {
            const int y = t / TPR, ch = t % TPR;
            if (4 * ch < width)
                *reinterpret_cast<int4*>(sm_cdt + y * CW + 4 * ch) = *reinterpret_cast<const int4*>(P.in + base + (int64_t)y * P.inner + 4 * ch);
        }
    } else {
        for (int t = threadIdx.x; t < n * CW; t += blockDim.x) {
            const int y = t / CW, x = t % CW;
            if (x < width) sm_cdt[y * CW + x] = P.in[base + (int64_t)y * P.inner + x];
        }
    }
    __syncthreads();
    constexpr int GPW = 32 / CW;  // row groups a warp works on at a time
    const int lane = threadIdx.x & (CW - 1), sub = (threadIdx.x & 31) / CW;
    const int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    if (lane >= width) return;
    auto op = [](int v, int d) { return CHESS ? max(v, d) : v + d; };
    for (int y0 = (warp * GPW + sub) * 4; y0 < n; y0 += nwarps * GPW * 4) {
        int k[4], best[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) k[i] = y0 + i < n ? sm_cdt[(y0 + i) * CW + lane] : kBig;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            best[i] = k[i];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (j != i) best[i] = min(best[i], op(k[j], i > j ? i - j : j - i));
            if (y0 + i >= n) best[i] = 0;
        }
        int mx = max(max(best[0], best[1]), max(best[2], best[3]));
        int lo = y0 - 1, hi = y0 + 4;
        for (int d = 1; d < mx && (lo >= 0 || hi < n); ++d, --lo, ++hi) {
            const int vlo = lo >= 0 ? sm_cdt[lo * CW + lane] : kBig;
            const int vhi = hi < n ? sm_cdt[hi * CW + lane] : kBig;
#pragma unroll
            for (int i = 0; i < 4; ++i) best[i] = min(best[i], min(op(vlo, d + i), op(vhi, d + 3 - i)));
            mx = max(max(best[0], best[1]), max(best[2], best[3]));
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (y0 + i < n) P.out[base + (int64_t)(y0 + i) * P.inner + lane] = (P.last && best[i] >= kBig) ? -1 : best[i];
    }
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
