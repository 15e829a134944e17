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

// ---- the first two axes on 16-bit values ----
// Distances along two axes of up to 1024 voxels each stay below 2^14, so the first pass hands 16-bit values to the
// second one (half the scratch traffic), and the second pass runs as sweeps in registers (below).  "No background
// seen" is kNone16 and every value at or above it means the same (adding distances to it stays below 2^16).
constexpr int kNone16 = 0xC000;

struct Row16Params {
    const uint8_t* mask;
    uint16_t* out;
    int64_t rows;
    int n0;          // voxels per row: a multiple of 4 (and of 32 unless the rows are at least 64 voxels long)
    int words;       // 32-voxel words per row, the last one possibly ragged (1 .. 32); the output rows have 32 words voxels
    uint16_t* edge;  // optional (rows, nb, 2): the values of columns 128 k - 1 and 128 k, k = 1 .. nb, for the pinned columns
    int nb;          // boundaries between groups of 128 columns (words / 4 rounded up, minus 1)
};

__device__ __forceinline__ uint32_t cdt_nonzero_bits4(uint32_t v) {
    const uint32_t m = (((v & 0x7f7f7f7fu) + 0x7f7f7f7fu) | v) & 0x80808080u;  // 0x80 in every nonzero byte
    return (((m >> 7) * 0x00204081u) >> 21) & 0xfu;
}

// First axis, rows of up to 1024 voxels (a multiple of 32, or of 4 with a ragged last word).  A lane owns one word of
// 32 voxels (one 32-byte load, two 32-byte stores into rows padded to whole words); a warp holds 32 / words whole rows.  The nearest background voxel outside the lane's word
// comes from a ballot over the words that contain one and a shuffle of its position inside that word; inside the word
// the distances are two running counts over the 32 bits, left to right and right to left.
// FAST: rows of a multiple of 32 voxels in a 32-byte aligned mask (one 256-bit load per lane).
template <bool FAST>
__global__ void __launch_bounds__(256, 4) cdt_row16_kernel(const __grid_constant__ Row16Params P) {
    const int lane = threadIdx.x & 31;
    const int64_t gw = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int words = P.words, rpw = 32 / words;
    const int grp = lane / words, w = lane - grp * words;
    const int64_t row = gw * rpw + grp;
    const bool valid = grp < rpw && row < P.rows;
    uint32_t z = 0u;  // bit i: voxel i of the word is background
    if (valid) {
        uint32_t v[8];
        const uint8_t* src = P.mask + row * P.n0 + 32 * w;
        if (FAST) {
            asm volatile("ld.global.nc.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                         : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                         : "l"(src));
        } else {  // rows of a multiple of 4 voxels: 4-byte loads; voxels beyond the row count as foreground
#pragma unroll
            for (int i = 0; i < 8; ++i)
                v[i] = 32 * w + 4 * i < P.n0 ? __ldg(reinterpret_cast<const uint32_t*>(src) + i) : 0x01010101u;
        }
        uint32_t nzb = 0u;
#pragma unroll
        for (int i = 0; i < 8; ++i) nzb |= cdt_nonzero_bits4(v[i]) << (4 * i);
        z = ~nzb;
    }
    const uint32_t has = __ballot_sync(0xffffffffu, z != 0u);
    const int g0 = grp * words, g1 = g0 + words;  // lanes of this row
    const uint32_t in_row = (g1 >= 32 ? 0xffffffffu : (1u << g1) - 1u) & ~((1u << g0) - 1u);
    const uint32_t left = has & in_row & ((1u << lane) - 1u);
    const uint32_t right = has & in_row & ~(lane == 31 ? 0xffffffffu : (2u << lane) - 1u);
    const int hb = 31 - __clz(z), lb = __ffs(z) - 1;  // last / first background voxel of the own word
    const int wl = left ? 31 - __clz(left) : lane, wr = right ? __ffs(right) - 1 : lane;
    const int hbl = __shfl_sync(0xffffffffu, hb, wl), lbr = __shfl_sync(0xffffffffu, lb, wr);
    if (!valid) return;
    int f = left ? 32 * (lane - wl) - hbl - 1 : kNone16;    // distance of the voxel before the word to the background on its left
    int d[32];
    const uint32_t fg = ~z;  // bit i: voxel i is foreground; count = fg_i * (count + 1) is one multiply-add
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const int keep = (int)((fg >> i) & 1u);
        f = keep * f + keep;
        d[i] = f;
    }
    int b = right ? 32 * (wr - lane) + lbr - 32 : kNone16;  // the same for the voxel after the word, to the right
#pragma unroll
    for (int i = 31; i >= 0; --i) {  // a row without background leaves values just above kNone16: "no background" all the same
        const int keep = (int)((fg >> i) & 1u);
        b = keep * b + keep;
        d[i] = min(d[i], b);
    }
    if (P.edge) {  // the last column of a group of 128 and the first one of the next group
        if ((w & 3) == 3 && w + 1 < words) P.edge[(row * P.nb + (w >> 2)) * 2] = (uint16_t)d[31];
        if ((w & 3) == 0 && w > 0) P.edge[(row * P.nb + (w >> 2) - 1) * 2 + 1] = (uint16_t)d[0];
    }
    uint16_t* dst = P.out + (row * words + w) * 32;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        uint32_t o[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) o[i] = (uint32_t)d[16 * h + 2 * i] | ((uint32_t)d[16 * h + 2 * i + 1] << 16);
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                     :: "l"(dst + 16 * h), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7])
                     : "memory");
    }
}

__device__ __forceinline__ uint32_t cdt_both(int v) { return (uint32_t)v * 0x00010001u; }  // v in both halves

// g(y) = min_j max(col[j], |y - j|) for eight consecutive rows y0 .. y0 + 7 of a contiguous column (rows beyond n are
// left out), by a bounded outward scan (a candidate d rows away is worth at least d, so the scan ends once d reaches
// the largest of the minima): the minima as four pairs of 16-bit halves, so that one candidate row serves all eight with two packed instructions per pair
// (max(f, d + offset) as one add-max, then a three-input minimum over both sides), two distances per stop test.
__device__ __forceinline__ void cdt_chess_scan8(const uint16_t* col, const int y0, const int n, uint16_t* res) {
    int k[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) k[i] = y0 + i < n ? (int)col[y0 + i] : kNone16;
    uint32_t B[4];  // minima of rows (y0 + 2p, y0 + 2p + 1) in the (low, high) halves
#pragma unroll
    for (int p = 0; p < 4; ++p) B[p] = (uint32_t)k[2 * p] | ((uint32_t)k[2 * p + 1] << 16);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t V = cdt_both(k[j]);
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            const int d0 = 2 * p > j ? 2 * p - j : j - 2 * p, d1 = 2 * p + 1 > j ? 2 * p + 1 - j : j - 2 * p - 1;
            B[p] = __vminu2(B[p], __vmaxu2(V, (uint32_t)d0 | ((uint32_t)d1 << 16)));
        }
    }
#pragma unroll
    for (int p = 0; p < 4; ++p) {  // rows beyond the axis: finished from the start
        if (y0 + 2 * p >= n) B[p] = 0u;
        else if (y0 + 2 * p + 1 >= n) B[p] &= 0xffffu;
    }
    auto largest = [&]() {
        const uint32_t m = __vmaxu2(__vimax3_u16x2(B[0], B[1], B[2]), B[3]);
        return (int)max(m & 0xffffu, m >> 16);
    };
    // rows lo and hi, d rows beyond the first and the last of the eight: row y0 + i is d + i from lo and d + 7 - i from hi
    auto step = [&](int vlo, int vhi, int d) {
        const uint32_t VL = cdt_both(vlo), VH = cdt_both(vhi), D = cdt_both(d);
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            const uint32_t cl = (uint32_t)(2 * p) | ((uint32_t)(2 * p + 1) << 16);
            const uint32_t chh = (uint32_t)(7 - 2 * p) | ((uint32_t)(6 - 2 * p) << 16);
            B[p] = __vimin3_u16x2(B[p], __viaddmax_u16x2(D, cl, VL), __viaddmax_u16x2(D, chh, VH));
        }
    };
    int mx = largest();
    int lo = y0 - 1, hi = y0 + 8, d = 1;
    for (; d < mx && lo >= 1 && hi + 1 < n; d += 2, lo -= 2, hi += 2) {  // the second distance is a true candidate either way
        const int a0 = col[lo], a1 = col[lo - 1], b0 = col[hi], b1 = col[hi + 1];
        step(a0, b0, d);
        step(a1, b1, d + 1);
        mx = largest();
    }
    for (; d < mx && (lo >= 0 || hi < n); ++d, --lo, ++hi) {
        step(lo >= 0 ? (int)col[lo] : kNone16, hi < n ? (int)col[hi] : kNone16, d);
        mx = largest();
    }
#pragma unroll
    for (int i = 0; i < 8; ++i)
        if (y0 + i < n) res[y0 + i] = (uint16_t)((B[i >> 1] >> (16 * (i & 1))) & 0xffffu);
}

// ---- second axis as sweeps between pinned voxels ----
// Taxicab: g(y) = min_j f(j) + |y - j| is two running minima, a(y) = min(f(y), a(y-1) + 1) down the rows and the same
// upwards starting from a.  Chessboard: g(y) = min_j max(f(j), |y - j|) has no such form along a column alone (a
// farther row with a smaller value can take over again later), but because f is a distance along the rows (it changes
// by at most 1 between neighbouring columns) the result obeys the two-sweep recurrence of the chamfer transform across
// columns: a(y, x) = min(f(y, x), 1 + min(a(y-1, x-1), a(y-1, x), a(y-1, x+1))) down the rows, then the same upwards.
// A sweep over a whole axis is sequential, so the image is cut into pieces of 31 rows x 128 columns by voxels whose
// exact results are computed first, by bounded scans (a candidate d rows away is worth at least d): every 32nd row of
// the axis and its last row, and for the chessboard metric the two columns at every boundary between groups of 128
// columns (cdt_pins_kernel; 3 % + 1.6 % of the voxels).  Every shortest path from a background voxel to a voxel of a
// piece either stays inside the piece or crosses a pinned voxel, whose exact value continues it, so the pieces are
// independent: cdt_sweep_kernel gives one warp a piece (a lane holds four neighbouring columns as the halves of two
// registers), loads its 31 rows at once, sweeps down from the pinned row above with the results kept in registers
// and up from the piece's own pinned row, writing the int32 output.  Work per voxel does not grow with the distances.
constexpr int kSegRows = 32;

struct SweepParams {
    const uint16_t* f;   // (slabs, n, inner): values of the first pass
    const uint16_t* edge;// (slabs, n, groups - 1, 2): the same at columns 128 k - 1 and 128 k, written by the first pass
    uint16_t* pd;        // (slabs, segs, inner): results of the pinned rows
    uint16_t* hd;        // (slabs, groups - 1, 2, n): results of the pinned columns 128 k - 1 and 128 k
    int32_t* out;
    int64_t slabs;
    int inner, n, segs, groups;
    int fpitch;          // voxels per row of f and pd (inner rounded up to a multiple of 32)
    int last;            // last pass: "no background" becomes -1 (else kBig for the next pass)
};

// Pinned rows: one lane per pair of neighbouring columns, a bounded outward scan along the axis through global memory
// (rows of pairs are contiguous: a warp reads 128 bytes per candidate row), eight distances per stop test.
template <bool CHESS>
__device__ __forceinline__ void cdt_pin_rows(const SweepParams& P, const int64_t t) {
    const int pairs = P.fpitch >> 1;
    if (t >= P.slabs * P.segs * pairs) return;
    const int x2 = (int)(t % pairs), k = (int)((t / pairs) % P.segs);
    const int64_t slab = t / ((int64_t)pairs * P.segs);
    const int n = P.n, y = min(n, (k + 1) * kSegRows) - 1;
    const uint32_t* col = reinterpret_cast<const uint32_t*>(P.f + slab * (int64_t)n * P.fpitch) + x2;
    const uint32_t none2 = cdt_both(kNone16);
    uint32_t best = col[(int64_t)y * pairs];
    int mx = (int)max(best & 0xffffu, best >> 16);
    auto cand = [&](uint32_t v, int d) { return CHESS ? __vmaxu2(v, cdt_both(d)) : v + cdt_both(d); };
    for (int d = 1; d < mx && (y - d >= 0 || y + d < n); d += 8) {  // sixteen loads in flight
        uint32_t a[8], b[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            a[i] = y - d - i >= 0 ? col[(int64_t)(y - d - i) * pairs] : none2;
            b[i] = y + d + i < n ? col[(int64_t)(y + d + i) * pairs] : none2;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) best = __vimin3_u16x2(best, cand(a[i], d + i), cand(b[i], d + i));
        mx = (int)max(best & 0xffffu, best >> 16);
    }
    reinterpret_cast<uint32_t*>(P.pd)[t] = __vminu2(best, none2);
}

// Blocks below row_blocks take 256 lanes of the pinned rows each; every further block takes one boundary between
// groups of 128 columns (chessboard only): the two columns beside it (gathered by the first pass) are staged in shared
// memory and scanned eight rows per lane.
template <bool CHESS>
__global__ void __launch_bounds__(256) cdt_pins_kernel(const __grid_constant__ SweepParams P, const unsigned row_blocks) {
    extern __shared__ __align__(16) uint16_t sm_pc[];  // [2][n] (column blocks)
    if (blockIdx.x < row_blocks) {
        cdt_pin_rows<CHESS>(P, (int64_t)blockIdx.x * 256 + threadIdx.x);
        return;
    }
    const int n = P.n, nb = P.groups - 1;
    const unsigned cb = blockIdx.x - row_blocks;
    const int k = (int)(cb % nb);
    const int64_t slab = cb / nb;
    const uint32_t* src = reinterpret_cast<const uint32_t*>(P.edge) + slab * (int64_t)n * nb + k;  // both columns of a row as one word
#pragma unroll 4
    for (int y = threadIdx.x; y < n; y += 256) {
        const uint32_t v = src[(int64_t)y * nb];
        sm_pc[y] = (uint16_t)(v & 0xffffu);
        sm_pc[n + y] = (uint16_t)(v >> 16);
    }
    __syncthreads();
    const int groups8 = (n + 7) >> 3;
    uint16_t* dst = P.hd + (slab * nb + k) * 2 * (int64_t)n;
    for (int t = threadIdx.x; t < 2 * groups8; t += 256) {
        const int side = t >= groups8;
        cdt_chess_scan8(sm_pc + side * n, (t - side * groups8) * 8, n, dst + side * n);
    }
}

template <bool CHESS>
__global__ void __launch_bounds__(128) cdt_sweep_kernel(const __grid_constant__ SweepParams P) {
    const int lane = threadIdx.x & 31;
    const int64_t gw = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (gw >= P.slabs * P.segs * P.groups) return;  // the whole warp
    const int g = (int)(gw % P.groups), k = (int)((gw / P.groups) % P.segs);
    const int64_t slab = gw / ((int64_t)P.groups * P.segs);
    const int n = P.n, inner = P.inner, c = 128 * g + 4 * lane;
    const bool act = c < inner;
    const int y0 = k * kSegRows, rp = min(n, y0 + kSegRows) - 1, cnt = rp - y0;  // swept rows y0 .. rp - 1
    const uint2 none2 = make_uint2(cdt_both(kNone16), cdt_both(kNone16));
    const int fp = P.fpitch;
    const uint16_t* fcol = P.f + slab * (int64_t)n * fp + (act ? c : 0);
    const uint16_t* pdk = P.pd + (slab * P.segs + k) * (int64_t)fp + (act ? c : 0);
    const uint16_t* hl = CHESS && g > 0 ? P.hd + ((slab * (P.groups - 1) + g - 1) * 2 + 0) * (int64_t)n : nullptr;
    const uint16_t* hr = CHESS && g + 1 < P.groups ? P.hd + ((slab * (P.groups - 1) + g) * 2 + 1) * (int64_t)n : nullptr;
    int32_t* out = P.out + slab * (int64_t)n * inner + (act ? c : 0);
    const int none_out = P.last ? -1 : kBig;
    auto put = [&](int y, uint2 v) {
        int r[4] = {(int)(v.x & 0xffffu), (int)(v.x >> 16), (int)(v.y & 0xffffu), (int)(v.y >> 16)};
#pragma unroll
        for (int i = 0; i < 4; ++i) r[i] = r[i] >= kNone16 ? none_out : r[i];
        if (act) *reinterpret_cast<int4*>(out + (int64_t)y * inner) = make_int4(r[0], r[1], r[2], r[3]);
    };
    // every row of the piece in flight at once
    uint2 a[kSegRows - 1];
#pragma unroll
    for (int i = 0; i < kSegRows - 1; ++i)
        a[i] = i < cnt && act ? *reinterpret_cast<const uint2*>(fcol + (int64_t)(y0 + i) * fp) : none2;
    // results of the pinned columns beside the piece: lane i holds row y0 - 1 + i, row y0 + 31 apart
    int hlv = kNone16, hrv = kNone16, hl_last = kNone16, hr_last = kNone16;
    if (CHESS) {
        const int yh = y0 - 1 + lane;
        if (hl && yh >= 0 && yh < n) hlv = hl[yh];
        if (hr && yh >= 0 && yh < n) hrv = hr[yh];
        if (hl && y0 + 31 < n) hl_last = hl[y0 + 31];
        if (hr && y0 + 31 < n) hr_last = hr[y0 + 31];
    }
    // one row of the recurrence: prev = the row before (after), ih = its place among the rows of the pinned columns
    auto relax = [&](uint2 prev, uint2 f, int ih) {
        uint2 r;
        if (CHESS) {
            uint32_t pl = __shfl_up_sync(0xffffffffu, prev.y, 1), pr = __shfl_down_sync(0xffffffffu, prev.x, 1);
            const int l_edge = ih < 32 ? __shfl_sync(0xffffffffu, hlv, ih & 31) : hl_last;
            const int r_edge = ih < 32 ? __shfl_sync(0xffffffffu, hrv, ih & 31) : hr_last;
            if (lane == 0) pl = (uint32_t)l_edge << 16;
            if (lane == 31) pr = (uint32_t)r_edge;
            const uint32_t L0 = __byte_perm(pl, prev.x, 0x5432), M = __byte_perm(prev.x, prev.y, 0x5432), R1 = __byte_perm(prev.y, pr, 0x5432);
            r.x = __viaddmin_u16x2(__vimin3_u16x2(L0, prev.x, M), 0x00010001u, f.x);
            r.y = __viaddmin_u16x2(__vimin3_u16x2(M, prev.y, R1), 0x00010001u, f.y);
        } else {
            r.x = __viaddmin_u16x2(prev.x, 0x00010001u, f.x);
            r.y = __viaddmin_u16x2(prev.y, 0x00010001u, f.y);
        }
        return act ? r : none2;  // lanes beyond the row stay "no background" for their neighbours
    };
    uint2 prev = act && k > 0 ? *reinterpret_cast<const uint2*>(pdk - fp) : none2;
#pragma unroll
    for (int i = 0; i < kSegRows - 1; ++i) {  // down from the pinned row above (row y0 + i - 1: place i)
        if (i < cnt) {
            a[i] = relax(prev, a[i], i);
            prev = a[i];
        }
    }
    prev = act ? *reinterpret_cast<const uint2*>(pdk) : none2;
    put(rp, prev);
#pragma unroll
    for (int i = kSegRows - 2; i >= 0; --i) {  // up from the own pinned row (row y0 + i + 1: place i + 2)
        if (i < cnt) {
            prev = relax(prev, a[i], i + 2);
            put(y0 + i, prev);
        }
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
