// Fast path for extents up to 128 and at most five processed axes.
//
// Carry layout ("entries"): after p + 1 processed axes every voxel holds one packed entry whose byte q
// (q <= p) is the signed offset  site_q - x_q  along processed axis q (plane order: contiguous axis
// first); 1, 2, 4 bytes for 1, 2, 3..4 axes.  Byte 0 == 0x80 marks "no site yet".  An entry of all
// zeros is a background voxel.  Entries make every load, gather and store of a voxel one access.
//
// Kernels (one thread block per (n_1 x n_0) plane, or per (n x 32 G) tile of a later axis):
//   plane_unit_kernel     unit sampling: the first-axis pass (four voxels per lane, ballot + shuffles)
//                         writes scan keys straight into a plane-wide shared tile, the second-axis pass
//                         scans it; 2-byte entries or the final outputs go to global memory.
//   plane_scaled_kernel   the same for sampling that becomes integer under a common scale.
//   plane_sampled_kernel  the same with float32 heights (any sampling).
//   plane_kernel          fallback for contiguous extents that are no multiple of 4 or unaligned input:
//                         byte loads, up to four ballot words per row, 32-column groups.
//   column_kernel         one further axis: a block stages a tile of entries in shared memory (TX
//                         consecutive positions of the contiguous `inner` index) and runs the pass on it.
//   column_scaled_kernel  the same in scaled integers.
//
// The pass along an axis (g_k(x) = min_j [ g_{k-1}(x with x_k := j) + (w_k (x_k - j))^2 ], paper
// Section 2.3.2) is taken voxel by voxel as an exact bounded scan instead of a sequential envelope
// sweep: starting from the voxel's own height, rows at distance d = 1, 2, .. on both sides are tried
// and the scan stops as soon as w^2 d^2 >= best, because no farther row can then be smaller.  The
// scan length is about the voxel's distance to the background along the axis -- short on real masks,
// and never more than the extent (<= 128).  Every voxel is independent, a warp works on 32 neighbouring
// columns of the same row (loads and stores are contiguous runs, neighbouring voxels have similar scan
// lengths), and background voxels (height 0) leave the loop at once.
//
// Integer heights (unit sampling, or scaled integers): the tile holds keys (height << s | row) so that
// one fused add-and-min instruction per candidate tracks value and site together, exactly; four
// consecutive rows of a column are scanned together so that every fetched candidate serves four voxels.
// Other sampling: heights are float32, the site is tracked by a compare and select.
#pragma once
#include "edt_common.cuh"

namespace tmedt {

template <int BYTES> struct EntryType;
template <> struct EntryType<1> { using type = uint8_t; };
template <> struct EntryType<2> { using type = uint16_t; };
template <> struct EntryType<4> { using type = uint32_t; };
__host__ __device__ constexpr int entry_bytes(int axes) { return axes <= 1 ? 1 : (axes == 2 ? 2 : 4); }

struct FastParams {
    const void* in;      // mask (plane kernel) or entries of K axes (column kernel)
    void* out;           // entries of K + 1 axes (unused when FINAL)
    int64_t outer;       // number of (outer) slabs; the array is (outer, n, inner)
    int64_t inner;
    int n;               // extent of the axis of this pass
    int n0;              // plane kernel: extent of the contiguous axis (== inner)
    float w2;            // squared sampling of this axis
    float w2p[4];        // squared sampling of the earlier axes (plane order)
    int si[4];           // scaled-integer mode: scale * w^2 of the earlier axes (exact integers)
    int sk;              // scaled-integer mode: scale * w^2 of this axis
    float inv_scale;     // scaled-integer mode: 1 / scale
    int value_carry;     // plane kernels, non-final: 0 = write entries; 2 / 4 = write the squared distance so far as
                         // uint16 / uint32 (all ones = no site), for the passes of edt_value.cuh
};

// add[d] = w^2 d^2 for the axis of the pass: float32 bits (sampled) or d^2 << shift (unit sampling keys).
struct ScanTab { uint32_t add[132]; };

constexpr uint32_t kNoneKey = 0xF0000000u;    // keys (value << 8 | row): values stay below 2^25
constexpr uint32_t kNoneKey16 = 0x80000000u;  // keys (value << 16 | row << 8 | offset): values stay below 2^15
#define TMEDT_INF (__int_as_float(0x7f800000))

__device__ __forceinline__ float small_int_to_float(int v) {  // exact for 0 <= v < 2^23, two full-rate ops
    return __int_as_float(v | 0x4B000000) - 8388608.0f;
}

__device__ __forceinline__ bool entry_none(uint32_t e) { return (e & 0xffu) == 0x80u; }

// Sum of the squared signed offsets of an entry (unused high bytes are zero): one 4-way byte dot product.
template <int K> __device__ __forceinline__ int entry_sumsq(uint32_t e) { return __dp4a((int)e, (int)e, 0); }

// Tile value the scan works on: unit sampling -> key (sum of squared offsets << 8 | row), none -> kNoneKey;
// otherwise the bits of the float32 height sum_q w_q^2 off_q^2, none -> +inf.
template <int K, bool UNIT>
__device__ __forceinline__ uint32_t scan_value(uint32_t e, int row, const float* w2p) {
    if (UNIT) return entry_none(e) ? kNoneKey : (((uint32_t)entry_sumsq<K>(e) << 8) | (uint32_t)row);
    if (entry_none(e)) return 0x7f800000u;
    int o = (int)(int8_t)(e & 0xff);
    float h = w2p[0] * small_int_to_float(o * o);
    if (K > 1) { o = (int)(int8_t)((e >> 8) & 0xff); h = fmaf(w2p[1], small_int_to_float(o * o), h); }
    if (K > 2) { o = (int)(int8_t)((e >> 16) & 0xff); h = fmaf(w2p[2], small_int_to_float(o * o), h); }
    if (K > 3) { o = (int)(int8_t)((e >> 24) & 0xff); h = fmaf(w2p[3], small_int_to_float(o * o), h); }
    return __float_as_uint(h);
}

// Where the results of one column (fixed thread <-> column) go.
template <int K, bool FINAL>
struct ColumnOut {
    typename EntryType<entry_bytes(K + 1)>::type* out;  // non-final: &out[row 0 of the column]
    float* dist; int64_t* sq; int64_t* idx;             // final: &buf[row 0 of the column] (idx: plane 0 of image)
    int64_t stride;      // distance between consecutive rows of the column, in voxels
    int64_t V;           // voxels per image (index-plane stride)
    int coord[4];        // own coordinates along the earlier planes
    int axis[5];         // spatial axis of plane q
    int ndim;
    bool dist_only;      // final: only out_dist was requested
    int64_t* ip[5];      // final: index plane of processed axis q (same row-0 origin as idx)
    bool simple_idx;     // final: every spatial axis is a processed axis (no extent-1 axes to fill with 0)
    bool flat;           // final: idx holds one value per voxel, the site's linear index inside the image
    int pst[5];          // flat: voxel stride of plane q inside the image

    // call after idx, V, ndim and axis[] are set
    __device__ __forceinline__ void init_index_planes(const EpilogueParams& ep) {
#pragma unroll
        for (int q = 0; q <= K; ++q) ip[q] = idx ? idx + (int64_t)axis[q] * V : nullptr;
        simple_idx = ndim == K + 1;
        flat = ep.flat != 0;
#pragma unroll
        for (int q = 0; q <= K; ++q) pst[q] = (int)ep.pstride[q];
    }
};

__device__ __forceinline__ float fast_sqrt(float v) {
    float r;
    asm("sqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}

// Emits row y of a column given the chosen site row j (or none), the site's entry and the squared distance.
template <int K, bool FINAL, bool UNIT>
__device__ __forceinline__ void emit(const ColumnOut<K, FINAL>& o, int y, int j, uint32_t e, float sqv, bool none) {
    const int64_t p = (int64_t)y * o.stride;
    if (!FINAL) {
        using EO = typename EntryType<entry_bytes(K + 1)>::type;
        const uint32_t v = none ? 0x80u : (e | ((uint32_t)((j - y) & 0xff) << (8 * (K & 3))));
        o.out[p] = (EO)v;
        return;
    }
    // sqv is exact for unit sampling (an integer below 2^24); the hardware root's relative error of about
    // 1e-7 is a hundred times inside the 1e-5 bar on distances.
    const float dv = none ? TMEDT_INF : fast_sqrt(sqv);
    if (o.dist_only) { o.dist[p] = dv; return; }
    if (o.dist) __stcs(o.dist + p, dv);
    if (none) {
        if (o.sq) o.sq[p] = INT64_MAX;
        if (o.idx && o.flat) o.idx[p] = -1;
        else if (o.idx)
            for (int a = 0; a < o.ndim; ++a) o.idx[(int64_t)a * o.V + p] = -1;
        return;
    }
    if (o.sq) o.sq[p] = (int64_t)sqv;  // unit sampling only
    if (o.idx && o.flat) {
        int f = j * o.pst[K];
#pragma unroll
        for (int q = 0; q < K; ++q) f += (o.coord[q] + (int)(int8_t)((e >> (8 * q)) & 0xff)) * o.pst[q];
        o.idx[p] = (int64_t)f;
    } else if (o.idx && o.simple_idx) {
        // one store per processed axis: own coordinate + offset (coordinates are non-negative)
#pragma unroll
        for (int q = 0; q < K; ++q)
            __stcs(reinterpret_cast<long long*>(o.ip[q] + p), (long long)(uint32_t)(o.coord[q] + (int)(int8_t)((e >> (8 * q)) & 0xff)));
        __stcs(reinterpret_cast<long long*>(o.ip[K] + p), (long long)(uint32_t)j);
    } else if (o.idx) {
        int off[5];
#pragma unroll
        for (int q = 0; q < K; ++q) off[q] = (int)(int8_t)((e >> (8 * q)) & 0xff);
        off[K] = j - y;
        // axes of extent 1 keep index 0; processed axes get own coordinate + offset
        for (int a = 0; a < o.ndim; ++a) {
            int64_t val = 0;
#pragma unroll
            for (int q = 0; q <= K; ++q)
                if (o.axis[q] == a) val = (int64_t)((q == K ? y : o.coord[q]) + off[q]);
            o.idx[(int64_t)a * o.V + p] = val;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Bounded scans of one voxel (row y of the column col[row * VS]).  All lanes of a warp share y, so the
// loop bounds are warp-uniform; lanes leave individually once add[d] >= best.
// ---------------------------------------------------------------------------------------------
// Unit sampling: keys carry the site, one fused add-min per candidate.
template <int VS>
__device__ __forceinline__ uint32_t scan_keys(const uint32_t* __restrict__ col, int n, int y, const ScanTab& tab) {
    uint32_t best = col[y * VS];
    const int up = y, dn = n - 1 - y, m = min(up, dn);
    const uint32_t* plo = col + (y - 1) * VS;
    const uint32_t* phi = col + (y + 1) * VS;
    int d = 1;
    for (; d + 1 <= m; d += 2) {
        const uint32_t a0 = tab.add[d], a1 = tab.add[d + 1];
        if (a0 >= best) return best;
        best = __viaddmin_u32(plo[0], a0, best);
        best = __viaddmin_u32(phi[0], a0, best);
        best = __viaddmin_u32(plo[-VS], a1, best);
        best = __viaddmin_u32(phi[VS], a1, best);
        plo -= 2 * VS; phi += 2 * VS;
    }
    if (d <= m) {
        const uint32_t a0 = tab.add[d];
        if (a0 >= best) return best;
        best = __viaddmin_u32(plo[0], a0, best);
        best = __viaddmin_u32(phi[0], a0, best);
        plo -= VS; phi += VS; ++d;
    }
    if (up > dn) {
        for (; d <= up; ++d, plo -= VS) {
            const uint32_t a0 = tab.add[d];
            if (a0 >= best) return best;
            best = __viaddmin_u32(plo[0], a0, best);
        }
    } else {
        for (; d <= dn; ++d, phi += VS) {
            const uint32_t a0 = tab.add[d];
            if (a0 >= best) return best;
            best = __viaddmin_u32(phi[0], a0, best);
        }
    }
    return best;
}

// Unit sampling, R consecutive rows y0 .. y0+R-1 of one column at once: every row fetched from the tile
// serves all R voxels (each with its own addend), which divides the shared-memory loads and the loop
// overhead per voxel by R.  Rows beyond the column end get best = 0 and are not emitted by the caller.
// wk: integer weight of the axis (1 for unit sampling); addends are wk * t^2 << SH.
template <int VS, int R, int SH = 8>
__device__ __forceinline__ void scan_keys_group(const uint32_t* __restrict__ col, int n, int y0, uint32_t (&best)[R],
                                                const uint32_t wk = 1u) {
    // "no site" key: above every real key, and adding any addend to it must not wrap around
    constexpr uint32_t NONE = SH == 8 ? kNoneKey : kNoneKey16;
    uint32_t k[R];
#pragma unroll
    for (int i = 0; i < R; ++i) k[i] = y0 + i < n ? col[(y0 + i) * VS] : NONE;
    if (SH == 0) {  // plain values: a group of background voxels is all zeros
        uint32_t any = k[0];
#pragma unroll
        for (int i = 1; i < R; ++i) any |= k[i];
        if (any == 0u) {
#pragma unroll
            for (int i = 0; i < R; ++i) best[i] = 0u;
            return;
        }
    }
#pragma unroll
    for (int i = 0; i < R; ++i) {
        best[i] = k[i];
#pragma unroll
        for (int j = 0; j < R; ++j)
            if (j != i) best[i] = __viaddmin_u32(k[j], (wk * (uint32_t)((i - j) * (i - j))) << SH, best[i]);
        if (y0 + i >= n) best[i] = 0u;
    }
    uint32_t mx = best[0];
#pragma unroll
    for (int i = 1; i < R; ++i) mx = max(mx, best[i]);
    if (mx < (1u << SH)) return;  // a group of background voxels
    const int dsafe = min(y0, n - R - y0);  // steps for which both outer rows exist
    int d = 1;
    // The first W steps as straight-line code with constant addends, no stop tests and no loop state: most
    // groups of real masks are finished by then (trying a few rows too many does not change the minimum).
    constexpr int W = 4;
    if (dsafe >= W) {
#pragma unroll
        for (int s = 1; s <= W; ++s) {
            const uint32_t vlo = col[(y0 - s) * VS], vhi = col[(y0 + R - 1 + s) * VS];
#pragma unroll
            for (int i = 0; i < R; ++i) {
                best[i] = __viaddmin_u32(vlo, (wk * (uint32_t)((s + i) * (s + i))) << SH, best[i]);
                best[i] = __viaddmin_u32(vhi, (wk * (uint32_t)((s + R - 1 - i) * (s + R - 1 - i))) << SH, best[i]);
            }
        }
        d = W + 1;
        mx = best[0];
#pragma unroll
        for (int i = 1; i < R; ++i) mx = max(mx, best[i]);
        if ((wk * (uint32_t)(d * d)) << SH >= mx) return;
    }
    uint32_t a[R];  // a[i] = (d + i)^2 << SH
#pragma unroll
    for (int i = 0; i < R; ++i) a[i] = (wk * (uint32_t)((d + i) * (d + i))) << SH;
    const uint32_t* plo = col + (y0 - d) * VS;
    const uint32_t* phi = col + (y0 + R - 1 + d) * VS;
    // interior steps, two at a time: both rows exist on both sides, no bounds tests, one stop test per pair
    for (; d + 1 <= dsafe && a[0] < mx; d += 2, plo -= 2 * VS, phi += 2 * VS) {
        const uint32_t vlo0 = plo[0], vhi0 = phi[0], vlo1 = plo[-VS], vhi1 = phi[VS];
        const uint32_t aR = (wk * (uint32_t)((d + R) * (d + R))) << SH;  // addend of distance d + R
#pragma unroll
        for (int i = 0; i < R; ++i) {
            best[i] = __viaddmin_u32(vlo0, a[i], best[i]);
            best[i] = __viaddmin_u32(vhi0, a[R - 1 - i], best[i]);
        }
#pragma unroll
        for (int i = 0; i < R; ++i) {  // step d + 1: distances (d + 1 + i) and (d + 1 + R - 1 - i)
            best[i] = __viaddmin_u32(vlo1, i + 1 < R ? a[i + 1] : aR, best[i]);
            best[i] = __viaddmin_u32(vhi1, R - i < R ? a[R - i] : aR, best[i]);
        }
        mx = best[0];
#pragma unroll
        for (int i = 1; i < R; ++i) mx = max(mx, best[i]);
#pragma unroll
        for (int i = 0; i + 2 < R; ++i) a[i] = a[i + 2];
        a[R - 2] = aR;
        a[R - 1] = (wk * (uint32_t)((d + R + 1) * (d + R + 1))) << SH;
    }
    for (; d <= dsafe && a[0] < mx; ++d, plo -= VS, phi += VS) {
        const uint32_t vlo = plo[0], vhi = phi[0];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            best[i] = __viaddmin_u32(vlo, a[i], best[i]);
            best[i] = __viaddmin_u32(vhi, a[R - 1 - i], best[i]);
        }
        mx = best[0];
#pragma unroll
        for (int i = 1; i < R; ++i) mx = max(mx, best[i]);
#pragma unroll
        for (int i = 0; i + 1 < R; ++i) a[i] = a[i + 1];
        a[R - 1] = (wk * (uint32_t)((d + R) * (d + R))) << SH;
    }
    // steps that reach past one end of the column
    int lo = y0 - d, hi = y0 + R - 1 + d;
    for (; a[0] < mx; ++d, --lo, ++hi, plo -= VS, phi += VS) {
        if (lo < 0 && hi >= n) break;
        if (lo >= 0) {
            const uint32_t v = plo[0];
#pragma unroll
            for (int i = 0; i < R; ++i) best[i] = __viaddmin_u32(v, a[i], best[i]);
        }
        if (hi < n) {
            const uint32_t v = phi[0];
#pragma unroll
            for (int i = 0; i < R; ++i) best[i] = __viaddmin_u32(v, a[R - 1 - i], best[i]);
        }
        mx = best[0];
#pragma unroll
        for (int i = 1; i < R; ++i) mx = max(mx, best[i]);
#pragma unroll
        for (int i = 0; i + 1 < R; ++i) a[i] = a[i + 1];
        a[R - 1] = (wk * (uint32_t)((d + R) * (d + R))) << SH;
    }
}

// Float heights.  ARG: also returns the distance bd (0 = own row) at which the minimum was found.
template <int VS, bool ARG>
__device__ __forceinline__ float scan_heights(const uint32_t* __restrict__ col, int n, int y, const ScanTab& tab,
                                              int& bd) {
    float best = __uint_as_float(col[y * VS]);
    bd = 0;
    const int up = y, dn = n - 1 - y, m = min(up, dn);
    const uint32_t* plo = col + (y - 1) * VS;
    const uint32_t* phi = col + (y + 1) * VS;
    int d = 1;
    for (; d + 1 <= m; d += 2) {
        const float a0 = __uint_as_float(tab.add[d]), a1 = __uint_as_float(tab.add[d + 1]);
        if (a0 >= best) return best;
        const float c0 = fminf(__uint_as_float(plo[0]), __uint_as_float(phi[0])) + a0;
        const float c1 = fminf(__uint_as_float(plo[-VS]), __uint_as_float(phi[VS])) + a1;
        if (ARG) {
            if (c0 < best) { best = c0; bd = d; }
            if (c1 < best) { best = c1; bd = d + 1; }
        } else {
            best = fminf(best, fminf(c0, c1));
        }
        plo -= 2 * VS; phi += 2 * VS;
    }
    if (d <= m) {
        const float a0 = __uint_as_float(tab.add[d]);
        if (a0 >= best) return best;
        const float c0 = fminf(__uint_as_float(plo[0]), __uint_as_float(phi[0])) + a0;
        if (ARG) { if (c0 < best) { best = c0; bd = d; } } else best = fminf(best, c0);
        plo -= VS; phi += VS; ++d;
    }
    if (up > dn) {
        for (; d <= up; ++d, plo -= VS) {
            const float a0 = __uint_as_float(tab.add[d]);
            if (a0 >= best) return best;
            const float c0 = __uint_as_float(plo[0]) + a0;
            if (ARG) { if (c0 < best) { best = c0; bd = d; } } else best = fminf(best, c0);
        }
    } else {
        for (; d <= dn; ++d, phi += VS) {
            const float a0 = __uint_as_float(tab.add[d]);
            if (a0 >= best) return best;
            const float c0 = __uint_as_float(phi[0]) + a0;
            if (ARG) { if (c0 < best) { best = c0; bd = d; } } else best = fminf(best, c0);
        }
    }
    return best;
}

// Scan of one voxel followed by its output.  ent[row * ES] are the entries of the column.
template <int K, bool FINAL, bool UNIT, int VS, typename ET>
__device__ __forceinline__ void scan_voxel(const uint32_t* __restrict__ col, const ET* __restrict__ ent, int ES, int n,
                                           int y, const ScanTab& tab, const ColumnOut<K, FINAL>& out) {
    int j;
    float sqv;
    bool none;
    if (UNIT) {
        const uint32_t best = scan_keys<VS>(col, n, y, tab);
        none = best >= kNoneKey;
        j = (int)(best & 0xffu);
        sqv = small_int_to_float((int)(best >> 8));
    } else if (FINAL) {
        // the site itself is only needed for index output: find it only then
        int bd;
        if (out.dist_only) {
            sqv = scan_heights<VS, false>(col, n, y, tab, bd);
            emit<K, FINAL, UNIT>(out, y, y, 0u, sqv, sqv == TMEDT_INF);
            return;
        }
        sqv = scan_heights<VS, true>(col, n, y, tab, bd);
        none = sqv == TMEDT_INF;
        j = y;
        if (bd > 0) {
            const float lo = bd <= y ? __uint_as_float(col[(y - bd) * VS]) : TMEDT_INF;
            const float hi = y + bd < n ? __uint_as_float(col[(y + bd) * VS]) : TMEDT_INF;
            j = lo <= hi ? y - bd : y + bd;
        }
    } else {
        int bd;
        sqv = scan_heights<VS, true>(col, n, y, tab, bd);
        none = sqv == TMEDT_INF;
        j = y;
        if (bd > 0) {
            const float lo = bd <= y ? __uint_as_float(col[(y - bd) * VS]) : TMEDT_INF;
            const float hi = y + bd < n ? __uint_as_float(col[(y + bd) * VS]) : TMEDT_INF;
            j = lo <= hi ? y - bd : y + bd;
        }
    }
    const uint32_t e = none ? 0u : (uint32_t)ent[j * ES];
    emit<K, FINAL, UNIT>(out, y, j, e, sqv, none);
}

// ---------------------------------------------------------------------------------------------
// First-axis pass of one row of a plane into shared memory: 1-byte offsets (or 0x80).
// One warp per row at a time; n0 <= 128, i.e. at most four ballot words.  All branch conditions are
// warp-uniform (they depend on the ballot words only).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void pass0_row_to_tile(const uint8_t* __restrict__ row, int n0, uint8_t* __restrict__ trow,
                                                  int lane) {
    unsigned Z[4];
    const int nw = (n0 + 31) >> 5;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        Z[w] = 0u;
        if (w < nw) {
            const int x = w * 32 + lane;
            const uint8_t b = x < n0 ? row[x] : (uint8_t)1;
            Z[w] = __ballot_sync(0xffffffffu, x < n0 && b == 0);
        }
    }
    int prevw[4], nextw[4];
    int last = -1000;
#pragma unroll
    for (int w = 0; w < 4; ++w) { prevw[w] = last; if (Z[w]) last = w * 32 + 31 - __clz(Z[w]); }
    int first = 1000;
#pragma unroll
    for (int w = 3; w >= 0; --w) { nextw[w] = first; if (Z[w]) first = w * 32 + __ffs(Z[w]) - 1; }
    const bool none = last < 0;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        if (w >= nw) break;
        const int x = w * 32 + lane;
        int off;
        if (none) off = -128;
        else if (Z[w] == 0xffffffffu) off = 0;
        else {
            const unsigned Zl = Z[w] & (0xffffffffu >> (31 - lane));
            const unsigned Zr = Z[w] >> lane;
            const int lp = Zl ? w * 32 + 31 - __clz(Zl) : prevw[w];
            const int rp = Zr ? x + __ffs(Zr) - 1 : nextw[w];
            off = (x - lp <= rp - x) ? (lp - x) : (rp - x);
        }
        if (x < n0) trow[x] = (uint8_t)(int8_t)off;
    }
}

template <bool FINAL, bool UNIT>
__global__ void __launch_bounds__(256) plane_kernel(const __grid_constant__ FastParams P,
                                                    const __grid_constant__ EpilogueParams ep,
                                                    const __grid_constant__ ScanTab tab) {
    extern __shared__ __align__(16) uint8_t sm_plane[];
    const int n0 = P.n0, n1 = P.n;
    const int tstride = (n0 + 15) & ~15;
    uint8_t* tile = sm_plane;                                                      // [n1][tstride] offsets
    uint32_t* val = reinterpret_cast<uint32_t*>(sm_plane + (((size_t)n1 * tstride + 15) & ~(size_t)15));  // [n1][32]
    const int64_t plane = blockIdx.x;  // planes = outer
    const uint8_t* src = reinterpret_cast<const uint8_t*>(P.in) + plane * (int64_t)n1 * n0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int y = warp; y < n1; y += nwarps) pass0_row_to_tile(src + (int64_t)y * n0, n0, tile + y * tstride, lane);
    __syncthreads();
    const float w2p[4] = {P.w2p[0], 0.f, 0.f, 0.f};
    const int ngroups = (n0 + 31) >> 5;
    for (int g = 0; g < ngroups; ++g) {
        const int c = g * 32 + lane;
        const bool live = c < n0;
        for (int y = warp; y < n1; y += nwarps)
            val[y * 32 + lane] = scan_value<1, UNIT>(live ? (uint32_t)tile[y * tstride + c] : 0x80u, y, w2p);
        __syncthreads();
        if (live) {
            ColumnOut<1, FINAL> out;
            out.stride = n0;
            if (!FINAL) {
                out.out = reinterpret_cast<uint16_t*>(P.out) + plane * (int64_t)n1 * n0 + c;
            } else {  // two processed axes: the plane is the image
                out.dist = ep.dist ? ep.dist + plane * ep.V + c : nullptr;
                out.sq = ep.sq ? ep.sq + plane * ep.V + c : nullptr;
                out.idx = ep.idx ? ep.idx + plane * ep.idx_planes * ep.V + c : nullptr;
                out.V = ep.V; out.ndim = ep.ndim;
                out.dist_only = ep.dist && !ep.sq && !ep.idx;
                out.coord[0] = c;
                out.axis[0] = ep.axis[0]; out.axis[1] = ep.axis[1];
                out.init_index_planes(ep);
            }
            if (UNIT && (!FINAL || out.dist_only)) {
                constexpr int R = 4;
                for (int y0 = warp * R; y0 < n1; y0 += nwarps * R) {
                    uint32_t best[R];
                    scan_keys_group<32, R>(val + lane, n1, y0, best);
#pragma unroll
                    for (int i = 0; i < R; ++i) {
                        const int y = y0 + i;
                        if (y >= n1) break;
                        const uint32_t b = best[i];
                        const bool none = b >= kNoneKey;
                        const int j = (int)(b & 0xffu);
                        const uint32_t e = none ? 0u : (uint32_t)tile[j * tstride + c];
                        emit<1, FINAL, true>(out, y, j, e, small_int_to_float((int)(b >> 8)), none);
                    }
                }
            } else {
                for (int y = warp; y < n1; y += nwarps)
                    scan_voxel<1, FINAL, UNIT, 32, uint8_t>(val + lane, tile + c, tstride, n1, y, tab, out);
            }
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------------
// Unit-sampling plane kernel: the first-axis pass writes scan keys straight into one tile that covers
// the whole plane, key = (off^2 << 16) | (row << 8) | (off & 0xff), so the second-axis scan needs no
// second tile and no gather: the chosen site's first-axis offset rides in the low byte of the key.
// First axis, one warp per row, four voxels per lane (one 32-bit load): zero bytes are found with a
// carry-free byte test, the nearest lanes holding a zero on either side with one ballot and clz / ffs,
// their zero positions with two shuffles; the four voxels of the lane are then finished in registers.
// Requires n0 % 4 == 0 (rows then start on 4-byte boundaries).
// ---------------------------------------------------------------------------------------------
// PLAIN: the key is off^2 alone (no row, no offset): for passes that carry values and need no site afterwards
template <bool PLAIN = false>
__device__ __forceinline__ void pass0_row_to_keys(const uint32_t v, int n0, int y, uint32_t* __restrict__ vrow,
                                                  int lane) {
    // v: the lane's four mask bytes of this row (0x01010101 for lanes beyond the row)
    const bool act = 4 * lane < n0;
    const uint32_t m = ~(((v & 0x7f7f7f7fu) + 0x7f7f7f7fu) | v) & 0x80808080u;  // 0x80 in every zero byte
    const unsigned any = __ballot_sync(0xffffffffu, m != 0u);  // inactive lanes hold foreground: m == 0
    // every lane of the warp stays in the shuffles below; only the final store is guarded
    uint4 keys;
    if (any == 0u) {  // no background in this row
        keys = make_uint4(kNoneKey16, kNoneKey16, kNoneKey16, kNoneKey16);
    } else if (PLAIN && __all_sync(0xffffffffu, m == 0x80808080u || !act)) {  // nothing but background: all zero
        keys = make_uint4(0u, 0u, 0u, 0u);
    } else {
        const int lzin = m ? (31 - __clz(m)) >> 3 : 0;   // highest zero byte of this lane
        const int fzin = m ? (__ffs(m) - 1) >> 3 : 0;    // lowest zero byte of this lane
        const unsigned ml = any & ((1u << lane) - 1u);
        const unsigned mr = lane < 31 ? any >> (lane + 1) : 0u;
        const int Ll = ml ? 31 - __clz(ml) : 0;
        const int Lr = mr ? lane + __ffs(mr) : 0;
        const int lz_l = __shfl_sync(0xffffffffu, lzin, Ll);
        const int fz_r = __shfl_sync(0xffffffffu, fzin, Lr);
        const int x0 = 4 * lane;
        int cur = ml ? 4 * Ll + lz_l : -1024;   // nearest zero left of this lane's voxels
        int dl[4], dr[4];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            if ((m >> (8 * b + 7)) & 1u) cur = x0 + b;
            dl[b] = x0 + b - cur;
        }
        cur = mr ? 4 * Lr + fz_r : 2048;        // nearest zero right of this lane's voxels
#pragma unroll
        for (int b = 3; b >= 0; --b) {
            if ((m >> (8 * b + 7)) & 1u) cur = x0 + b;
            dr[b] = cur - (x0 + b);
        }
        uint32_t kk[4];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int a = min(dl[b], dr[b]);
            const int off = dl[b] <= dr[b] ? -a : a;
            kk[b] = PLAIN ? (uint32_t)(a * a) : (((uint32_t)(a * a) << 16) | ((uint32_t)y << 8) | ((uint32_t)off & 0xffu));
        }
        keys = make_uint4(kk[0], kk[1], kk[2], kk[3]);
    }
    if (act) *reinterpret_cast<uint4*>(vrow + 4 * lane) = keys;
}

// VC: what a non-final pass writes: 0 = 2-byte entries, 2 / 4 = the squared distance so far as uint16 / uint32.
template <bool FINAL, int VS, int VC = 0>
__global__ void __launch_bounds__(256) plane_unit_kernel(const __grid_constant__ FastParams P,
                                                         const __grid_constant__ EpilogueParams ep) {
    extern __shared__ __align__(16) uint8_t sm_plane_u[];
    uint32_t* val = reinterpret_cast<uint32_t*>(sm_plane_u);  // [n1][VS]
    const int n0 = P.n0, n1 = P.n;
    const int64_t plane = blockIdx.x;
    const uint8_t* src = reinterpret_cast<const uint8_t*>(P.in) + plane * (int64_t)n1 * n0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    {
        // all loads of this warp's rows are issued before the first row is processed
        constexpr int MAXR = 16;  // rows per warp: 128 rows / 8 warps
        uint32_t rowv[MAXR];
        const bool act = 4 * lane < n0;
#pragma unroll
        for (int i = 0; i < MAXR; ++i) {
            const int y = warp + i * nwarps;
            rowv[i] = (act && y < n1) ? *reinterpret_cast<const uint32_t*>(src + y * n0 + 4 * lane) : 0x01010101u;
        }
#pragma unroll
        for (int i = 0; i < MAXR; ++i) {
            const int y = warp + i * nwarps;
            if (y < n1) pass0_row_to_keys<(VC != 0)>(rowv[i], n0, y, val + y * VS, lane);
        }
    }
    __syncthreads();
    constexpr int R = 4, CG = VS / 32;
    const int tasks = ((n1 + R - 1) / R) * CG;
    const bool dist_only = FINAL && ep.dist && !ep.sq && !ep.idx;
    for (int t = warp; t < tasks; t += nwarps) {
        const int cg = t % CG, y0 = (t / CG) * R;
        const int c = cg * 32 + lane;
        if (c >= n0) continue;
        uint32_t best[R];
        scan_keys_group<VS, R, VC != 0 ? 0 : 16>(val + c, n1, y0, best);
        const int64_t p0 = plane * (int64_t)n1 * n0 + (int64_t)y0 * n0 + c;
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int y = y0 + i;
            if (y >= n1) break;
            const uint32_t b = best[i];
            const bool none = b >= kNoneKey16;
            const int j = (int)((b >> 8) & 0xffu);
            if (!FINAL) {
                if (VC == 2) {
                    reinterpret_cast<uint16_t*>(P.out)[p0 + (int64_t)i * n0] = (uint16_t)(none ? 0xffffu : b);
                } else if (VC == 4) {
                    reinterpret_cast<uint32_t*>(P.out)[p0 + (int64_t)i * n0] = none ? 0xffffffffu : b;
                } else {
                    const uint32_t e = none ? 0x80u : ((b & 0xffu) | ((uint32_t)((j - y) & 0xff) << 8));
                    reinterpret_cast<uint16_t*>(P.out)[p0 + (int64_t)i * n0] = (uint16_t)e;
                }
            } else if (VC != 0) {  // last pass without index output: plain values
                if (ep.dist) __stcs(ep.dist + p0 + (int64_t)i * n0, none ? TMEDT_INF : fast_sqrt(small_int_to_float((int)b)));
                if (ep.sq) __stcs(reinterpret_cast<long long*>(ep.sq + p0 + (int64_t)i * n0), none ? (long long)INT64_MAX : (long long)b);
            } else if (dist_only) {
                ep.dist[p0 + (int64_t)i * n0] = none ? TMEDT_INF : fast_sqrt(small_int_to_float((int)(b >> 16)));
            } else {  // two processed axes: the plane is the image
                ColumnOut<1, true> out;
                out.stride = n0;
                out.dist = ep.dist ? ep.dist + plane * ep.V + c : nullptr;
                out.sq = ep.sq ? ep.sq + plane * ep.V + c : nullptr;
                out.idx = ep.idx ? ep.idx + plane * ep.idx_planes * ep.V + c : nullptr;
                out.V = ep.V; out.ndim = ep.ndim; out.dist_only = false;
                out.coord[0] = c;
                out.axis[0] = ep.axis[0]; out.axis[1] = ep.axis[1];
                out.init_index_planes(ep);
                emit<1, true, true>(out, y, j, b & 0xffu, small_int_to_float((int)(b >> 16)), none);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Sampled plane kernel (general sampling, n0 % 4 == 0): like the unit-sampling one, but the tile holds
// float32 heights w0^2 off^2 and a second, byte-sized tile keeps the first-axis offsets for the output.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void pass0_row_to_heights(const uint32_t v, int n0, float w2x, uint32_t* __restrict__ vrow,
                                                     uint8_t* __restrict__ drow, int lane) {
    const bool act = 4 * lane < n0;
    const uint32_t m = ~(((v & 0x7f7f7f7fu) + 0x7f7f7f7fu) | v) & 0x80808080u;  // 0x80 in every zero byte
    const unsigned any = __ballot_sync(0xffffffffu, m != 0u);
    uint4 hv;
    uint32_t dpack;
    if (any == 0u) {  // no background in this row
        hv = make_uint4(0x7f800000u, 0x7f800000u, 0x7f800000u, 0x7f800000u);
        dpack = 0x80808080u;
    } else {
        const int lzin = m ? (31 - __clz(m)) >> 3 : 0;
        const int fzin = m ? (__ffs(m) - 1) >> 3 : 0;
        const unsigned ml = any & ((1u << lane) - 1u);
        const unsigned mr = lane < 31 ? any >> (lane + 1) : 0u;
        const int Ll = ml ? 31 - __clz(ml) : 0;
        const int Lr = mr ? lane + __ffs(mr) : 0;
        const int lz_l = __shfl_sync(0xffffffffu, lzin, Ll);
        const int fz_r = __shfl_sync(0xffffffffu, fzin, Lr);
        const int x0 = 4 * lane;
        int cur = ml ? 4 * Ll + lz_l : -1024;
        int dl[4], dr[4];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            if ((m >> (8 * b + 7)) & 1u) cur = x0 + b;
            dl[b] = x0 + b - cur;
        }
        cur = mr ? 4 * Lr + fz_r : 2048;
#pragma unroll
        for (int b = 3; b >= 0; --b) {
            if ((m >> (8 * b + 7)) & 1u) cur = x0 + b;
            dr[b] = cur - (x0 + b);
        }
        uint32_t hh[4];
        dpack = 0u;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int a = min(dl[b], dr[b]);
            const int off = dl[b] <= dr[b] ? -a : a;
            hh[b] = __float_as_uint(w2x * small_int_to_float(a * a));
            dpack |= ((uint32_t)off & 0xffu) << (8 * b);
        }
        hv = make_uint4(hh[0], hh[1], hh[2], hh[3]);
    }
    if (act) {
        *reinterpret_cast<uint4*>(vrow + 4 * lane) = hv;
        *reinterpret_cast<uint32_t*>(drow + 4 * lane) = dpack;
    }
}

template <bool FINAL, int VS>
__global__ void __launch_bounds__(512) plane_sampled_kernel(const __grid_constant__ FastParams P,
                                                            const __grid_constant__ EpilogueParams ep,
                                                            const __grid_constant__ ScanTab tab) {
    extern __shared__ __align__(16) uint8_t sm_plane_s[];
    const int n0 = P.n0, n1 = P.n;
    uint32_t* val = reinterpret_cast<uint32_t*>(sm_plane_s);                 // [n1][VS] float32 heights
    uint8_t* dxt = sm_plane_s + (size_t)n1 * VS * 4;                         // [n1][VS] first-axis offsets
    const int64_t plane = blockIdx.x;
    const uint8_t* src = reinterpret_cast<const uint8_t*>(P.in) + plane * (int64_t)n1 * n0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    {
        constexpr int MAXR = 16;
        uint32_t rowv[MAXR];
        const bool act = 4 * lane < n0;
#pragma unroll
        for (int i = 0; i < MAXR; ++i) {
            const int y = warp + i * nwarps;
            rowv[i] = (act && y < n1) ? *reinterpret_cast<const uint32_t*>(src + y * n0 + 4 * lane) : 0x01010101u;
        }
#pragma unroll
        for (int i = 0; i < MAXR; ++i) {
            const int y = warp + i * nwarps;
            if (y < n1) pass0_row_to_heights(rowv[i], n0, P.w2p[0], val + y * VS, dxt + y * VS, lane);
        }
    }
    __syncthreads();
    // a warp keeps one 32-column group and strides over the rows (nwarps is a multiple of VS / 32)
    constexpr int CG = VS / 32;
    const int cg = warp % CG, r0 = warp / CG, rstep = nwarps / CG;
    const int c = cg * 32 + lane;
    if (c >= n0) return;
    ColumnOut<1, FINAL> out;
    out.stride = n0;
    if (!FINAL) {
        out.out = reinterpret_cast<uint16_t*>(P.out) + plane * (int64_t)n1 * n0 + c;
    } else {  // two processed axes: the plane is the image
        out.dist = ep.dist ? ep.dist + plane * ep.V + c : nullptr;
        out.sq = nullptr;
        out.idx = ep.idx ? ep.idx + plane * ep.idx_planes * ep.V + c : nullptr;
        out.V = ep.V; out.ndim = ep.ndim;
        out.dist_only = ep.dist && !ep.idx;
        out.coord[0] = c;
        out.axis[0] = ep.axis[0]; out.axis[1] = ep.axis[1];
        out.init_index_planes(ep);
    }
    for (int y = r0; y < n1; y += rstep)
        scan_voxel<1, FINAL, false, VS, uint8_t>(val + c, dxt + c, VS, n1, y, tab, out);
}

template <int K, bool FINAL, bool UNIT, int TX>
__global__ void __launch_bounds__(256) column_kernel(const __grid_constant__ FastParams P,
                                                     const __grid_constant__ EpilogueParams ep,
                                                     const __grid_constant__ ScanTab tab,
                                                     const int tiles_per_slab) {
    using EI = typename EntryType<entry_bytes(K)>::type;
    extern __shared__ __align__(16) uint8_t sm_col[];
    constexpr int G = TX / 32;
    const int n = P.n;
    uint32_t* val = reinterpret_cast<uint32_t*>(sm_col);                  // [n][TX]
    EI* tile = reinterpret_cast<EI*>(sm_col + (size_t)n * TX * 4);        // [n][TX]
    const int64_t slab = blockIdx.x / tiles_per_slab;
    const int64_t i0 = (int64_t)(blockIdx.x - slab * tiles_per_slab) * TX;
    const int width = (int)min((int64_t)TX, P.inner - i0);
    const EI* src = reinterpret_cast<const EI*>(P.in) + slab * (int64_t)n * P.inner + i0;
    const float w2p[4] = {P.w2p[0], P.w2p[1], P.w2p[2], P.w2p[3]};
    // stage entries and scan values: 16-byte chunks when rows are 16-byte aligned, single entries otherwise
    constexpr int PER16 = 16 / (int)sizeof(EI);
    if ((P.inner % PER16) == 0 && (width % PER16) == 0) {
        constexpr int FULL = TX / PER16;
        const int chunks = width / PER16;
        for (int t = threadIdx.x; t < n * chunks; t += blockDim.x) {
            const int y = chunks == FULL ? t / FULL : t / chunks, ch = t - y * chunks;
            const uint4 v = *reinterpret_cast<const uint4*>(src + (int64_t)y * P.inner + ch * PER16);
            *reinterpret_cast<uint4*>(tile + y * TX + ch * PER16) = v;
            const uint32_t wv[4] = {v.x, v.y, v.z, v.w};
            uint32_t sv[PER16];
#pragma unroll
            for (int i = 0; i < PER16; ++i) {
                const uint32_t word = wv[(i * (int)sizeof(EI)) >> 2];
                const uint32_t e = sizeof(EI) == 4 ? word
                                 : sizeof(EI) == 2 ? ((word >> (16 * (i & 1))) & 0xffffu)
                                                   : ((word >> (8 * (i & 3))) & 0xffu);
                sv[i] = scan_value<K, UNIT>(e, y, w2p);
            }
#pragma unroll
            for (int i = 0; i < PER16; i += 4)
                *reinterpret_cast<uint4*>(val + y * TX + ch * PER16 + i) = make_uint4(sv[i], sv[i + 1], sv[i + 2], sv[i + 3]);
        }
    } else {
        for (int t = threadIdx.x; t < n * width; t += blockDim.x) {
            const int y = t / width, x = t - y * width;
            const EI e = src[(int64_t)y * P.inner + x];
            tile[y * TX + x] = e;
            val[y * TX + x] = scan_value<K, UNIT>((uint32_t)e, y, w2p);
        }
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int g = warp % G, r0 = warp / G, rstep = nwarps / G;
    const int c = g * 32 + lane;
    if (c >= width) return;
    ColumnOut<K, FINAL> out;
    out.stride = P.inner;
    if (!FINAL) {
        using EO = typename EntryType<entry_bytes(K + 1)>::type;
        out.out = reinterpret_cast<EO*>(P.out) + slab * (int64_t)n * P.inner + i0 + c;
    } else {
        // last pass: the slab is the image; i0 + c enumerates the earlier planes, plane 0 fastest
        const int64_t v0 = i0 + c;
        out.dist = ep.dist ? ep.dist + slab * ep.V + v0 : nullptr;
        out.sq = ep.sq ? ep.sq + slab * ep.V + v0 : nullptr;
        out.idx = ep.idx ? ep.idx + slab * ep.idx_planes * ep.V + v0 : nullptr;
        out.V = ep.V; out.ndim = ep.ndim;
        out.dist_only = ep.dist && !ep.sq && !ep.idx;
        uint32_t rr = (uint32_t)v0;  // a position inside one image: below 2^31
#pragma unroll
        for (int q = 0; q < K; ++q) {
            const uint32_t nq = (uint32_t)ep.ext[q], hi = rr / nq;
            out.coord[q] = (int)(rr - hi * nq);
            rr = hi;
        }
#pragma unroll
        for (int q = 0; q <= K; ++q) out.axis[q] = ep.axis[q];
        out.init_index_planes(ep);
    }
    if (UNIT) {
        constexpr int R = 4;
        for (int y0 = r0 * R; y0 < n; y0 += rstep * R) {
            uint32_t best[R];
            scan_keys_group<TX, R>(val + c, n, y0, best);
#pragma unroll
            for (int i = 0; i < R; ++i) {
                const int y = y0 + i;
                if (y >= n) break;
                // no special case for background voxels: their key names their own row, whose entry is 0
                const uint32_t b = best[i];
                const bool none = b >= kNoneKey;
                const int j = (int)(b & 0xffu);
                const uint32_t e = none ? 0u : (uint32_t)tile[j * TX + c];
                emit<K, FINAL, true>(out, y, j, e, small_int_to_float((int)(b >> 8)), none);
            }
        }
    } else {
        for (int y = r0; y < n; y += rstep)
            scan_voxel<K, FINAL, UNIT, TX, EI>(val + c, tile + c, TX, n, y, tab, out);
    }
}

// ---------------------------------------------------------------------------------------------
// Scaled-integer mode.  When a common scale S makes every S * w_q^2 an integer (sampling given with a
// few decimals: 0.8, 1.25, 2.5 ..) and the largest possible value S * sum_q w_q^2 (n_q - 1)^2 stays below
// 2^24, the transform with that sampling is exact integer arithmetic again: keys are
// (S * height) << 7 | row, candidates are combined with the fused add-min, and four rows share every
// fetched candidate, exactly as for unit sampling.  Distances are sqrt(value / S).
// ---------------------------------------------------------------------------------------------
constexpr int kScaledShift = 7;

template <int K>
__device__ __forceinline__ uint32_t scaled_key(uint32_t e, int row, const int* si) {
    if (entry_none(e)) return kNoneKey16;
    int o = (int)(int8_t)(e & 0xff);
    int v = si[0] * o * o;
    if (K > 1) { o = (int)(int8_t)((e >> 8) & 0xff); v += si[1] * o * o; }
    if (K > 2) { o = (int)(int8_t)((e >> 16) & 0xff); v += si[2] * o * o; }
    if (K > 3) { o = (int)(int8_t)((e >> 24) & 0xff); v += si[3] * o * o; }
    return ((uint32_t)v << kScaledShift) | (uint32_t)row;
}

// Outputs of row y from a scaled key; ent[row * ES] are the entries of the column.
template <int K, bool FINAL, typename ET>
__device__ __forceinline__ void emit_scaled(const ColumnOut<K, FINAL>& out, const ET* __restrict__ ent, int ES, int y,
                                            uint32_t b, float inv_scale) {
    const bool none = b >= kNoneKey16;  // background voxels need no special case: their key names their own row
    const int j = (int)(b & ((1u << kScaledShift) - 1u));
    const uint32_t e = none ? 0u : (uint32_t)ent[j * ES];
    emit<K, FINAL, false>(out, y, j, e, __uint2float_rn(b >> kScaledShift) * inv_scale, none);  // values reach 2^24
}

// WITH_OFF: also write the signed first-axis offsets as bytes (needed only when offsets are carried or indexed)
template <bool WITH_OFF = true>
__device__ __forceinline__ void pass0_row_to_scaled_keys(const uint32_t v, int n0, int y, int s0,
                                                         uint32_t* __restrict__ vrow, uint8_t* __restrict__ drow,
                                                         int lane) {
    const bool act = 4 * lane < n0;
    const uint32_t m = ~(((v & 0x7f7f7f7fu) + 0x7f7f7f7fu) | v) & 0x80808080u;  // 0x80 in every zero byte
    const unsigned any = __ballot_sync(0xffffffffu, m != 0u);
    uint4 kv;
    uint32_t dpack;
    if (any == 0u) {  // no background in this row
        kv = make_uint4(kNoneKey16, kNoneKey16, kNoneKey16, kNoneKey16);
        dpack = 0x80808080u;
    } else if (__all_sync(0xffffffffu, m == 0x80808080u || !act)) {  // nothing but background: every distance is 0
        const uint32_t k0 = WITH_OFF ? (uint32_t)y : 0u;
        kv = make_uint4(k0, k0, k0, k0);
        dpack = 0u;
    } else {
        const int lzin = m ? (31 - __clz(m)) >> 3 : 0;
        const int fzin = m ? (__ffs(m) - 1) >> 3 : 0;
        const unsigned ml = any & ((1u << lane) - 1u);
        const unsigned mr = lane < 31 ? any >> (lane + 1) : 0u;
        const int Ll = ml ? 31 - __clz(ml) : 0;
        const int Lr = mr ? lane + __ffs(mr) : 0;
        const int lz_l = __shfl_sync(0xffffffffu, lzin, Ll);
        const int fz_r = __shfl_sync(0xffffffffu, fzin, Lr);
        const int x0 = 4 * lane;
        int cur = ml ? 4 * Ll + lz_l : -1024;
        int dl[4], dr[4];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            if ((m >> (8 * b + 7)) & 1u) cur = x0 + b;
            dl[b] = x0 + b - cur;
        }
        cur = mr ? 4 * Lr + fz_r : 2048;
#pragma unroll
        for (int b = 3; b >= 0; --b) {
            if ((m >> (8 * b + 7)) & 1u) cur = x0 + b;
            dr[b] = cur - (x0 + b);
        }
        uint32_t kk[4];
        dpack = 0u;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int a = min(dl[b], dr[b]);
            const int off = dl[b] <= dr[b] ? -a : a;
            // without offsets no site is needed afterwards: the key is the plain value, without row bits
            kk[b] = WITH_OFF ? (((uint32_t)(s0 * a * a) << kScaledShift) | (uint32_t)y) : (uint32_t)(s0 * a * a);
            if (WITH_OFF) dpack |= ((uint32_t)off & 0xffu) << (8 * b);
        }
        kv = make_uint4(kk[0], kk[1], kk[2], kk[3]);
    }
    if (act) {
        *reinterpret_cast<uint4*>(vrow + 4 * lane) = kv;
        if (WITH_OFF) *reinterpret_cast<uint32_t*>(drow + 4 * lane) = dpack;
    }
}

// VC: a non-final pass writes the scaled squared distance so far (uint32) instead of entries; no offsets are kept.
template <bool FINAL, int VS, bool VC = false>
__global__ void __launch_bounds__(512, VC ? 3 : 2) plane_scaled_kernel(const __grid_constant__ FastParams P,
                                                           const __grid_constant__ EpilogueParams ep) {
    extern __shared__ __align__(16) uint8_t sm_plane_i[];
    const int n0 = P.n0, n1 = P.n;
    uint32_t* val = reinterpret_cast<uint32_t*>(sm_plane_i);   // [n1][VS] keys
    uint8_t* dxt = sm_plane_i + (size_t)n1 * VS * 4;           // [n1][VS] first-axis offsets
    const int64_t plane = blockIdx.x;
    const uint8_t* src = reinterpret_cast<const uint8_t*>(P.in) + plane * (int64_t)n1 * n0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    {
        constexpr int MAXR = 16;
        uint32_t rowv[MAXR];
        const bool act = 4 * lane < n0;
#pragma unroll
        for (int i = 0; i < MAXR; ++i) {
            const int y = warp + i * nwarps;
            rowv[i] = (act && y < n1) ? *reinterpret_cast<const uint32_t*>(src + y * n0 + 4 * lane) : 0x01010101u;
        }
#pragma unroll
        for (int i = 0; i < MAXR; ++i) {
            const int y = warp + i * nwarps;
            if (y < n1) pass0_row_to_scaled_keys<!VC>(rowv[i], n0, y, P.si[0], val + y * VS, dxt + y * VS, lane);
        }
    }
    __syncthreads();
    constexpr int R = 4, CG = VS / 32;
    const int cg = warp % CG, r0 = warp / CG, rstep = nwarps / CG;
    const int c = cg * 32 + lane;
    if (c >= n0) return;
    ColumnOut<1, FINAL> out;
    out.stride = n0;
    if (!FINAL) {
        out.out = reinterpret_cast<uint16_t*>(P.out) + plane * (int64_t)n1 * n0 + c;
    } else {  // two processed axes: the plane is the image
        out.dist = ep.dist ? ep.dist + plane * ep.V + c : nullptr;
        out.sq = nullptr;
        out.idx = ep.idx ? ep.idx + plane * ep.idx_planes * ep.V + c : nullptr;
        out.V = ep.V; out.ndim = ep.ndim;
        out.dist_only = ep.dist && !ep.idx;
        out.coord[0] = c;
        out.axis[0] = ep.axis[0]; out.axis[1] = ep.axis[1];
        out.init_index_planes(ep);
    }
    for (int y0 = r0 * R; y0 < n1; y0 += rstep * R) {
        uint32_t best[R];
        scan_keys_group<VS, R, VC ? 0 : kScaledShift>(val + c, n1, y0, best, (uint32_t)P.sk);
#pragma unroll
        for (int i = 0; i < R; ++i) {
            if (y0 + i >= n1) break;
            if (!FINAL && VC) {
                const uint32_t b = best[i];
                reinterpret_cast<uint32_t*>(P.out)[plane * (int64_t)n1 * n0 + (int64_t)(y0 + i) * n0 + c] =
                    b >= kNoneKey16 ? 0xffffffffu : b;
            } else if (FINAL && VC) {  // last pass, distances only: plain values
                const uint32_t b = best[i];
                __stcs(ep.dist + plane * ep.V + (int64_t)(y0 + i) * n0 + c,
                       b >= kNoneKey16 ? TMEDT_INF : fast_sqrt(__uint2float_rn(b) * P.inv_scale));
            } else {
                emit_scaled<1, FINAL, uint8_t>(out, dxt + c, VS, y0 + i, best[i], P.inv_scale);
            }
        }
    }
}

template <int K, bool FINAL, int TX>
__global__ void __launch_bounds__(256) column_scaled_kernel(const __grid_constant__ FastParams P,
                                                            const __grid_constant__ EpilogueParams ep,
                                                            const int tiles_per_slab) {
    using EI = typename EntryType<entry_bytes(K)>::type;
    extern __shared__ __align__(16) uint8_t sm_col_i[];
    constexpr int G = TX / 32;
    const int n = P.n;
    uint32_t* val = reinterpret_cast<uint32_t*>(sm_col_i);               // [n][TX]
    EI* tile = reinterpret_cast<EI*>(sm_col_i + (size_t)n * TX * 4);     // [n][TX]
    const int64_t slab = blockIdx.x / tiles_per_slab;
    const int64_t i0 = (int64_t)(blockIdx.x - slab * tiles_per_slab) * TX;
    const int width = (int)min((int64_t)TX, P.inner - i0);
    const EI* src = reinterpret_cast<const EI*>(P.in) + slab * (int64_t)n * P.inner + i0;
    const int si[4] = {P.si[0], P.si[1], P.si[2], P.si[3]};
    constexpr int PER16 = 16 / (int)sizeof(EI);
    if ((P.inner % PER16) == 0 && width == TX) {  // full tile, 16-byte aligned rows
        constexpr int FULL = TX / PER16;
        for (int t = threadIdx.x; t < n * FULL; t += blockDim.x) {
            const int y = t / FULL, ch = t - y * FULL;
            const uint4 v = *reinterpret_cast<const uint4*>(src + (int64_t)y * P.inner + ch * PER16);
            *reinterpret_cast<uint4*>(tile + y * TX + ch * PER16) = v;
            const uint32_t wv[4] = {v.x, v.y, v.z, v.w};
            uint32_t sv[PER16];
#pragma unroll
            for (int i = 0; i < PER16; ++i) {
                const uint32_t word = wv[(i * (int)sizeof(EI)) >> 2];
                const uint32_t e = sizeof(EI) == 4 ? word
                                 : sizeof(EI) == 2 ? ((word >> (16 * (i & 1))) & 0xffffu)
                                                   : ((word >> (8 * (i & 3))) & 0xffu);
                sv[i] = scaled_key<K>(e, y, si);
            }
#pragma unroll
            for (int i = 0; i < PER16; i += 4)
                *reinterpret_cast<uint4*>(val + y * TX + ch * PER16 + i) = make_uint4(sv[i], sv[i + 1], sv[i + 2], sv[i + 3]);
        }
    } else {
        for (int t = threadIdx.x; t < n * width; t += blockDim.x) {
            const int y = t / width, x = t - y * width;
            const EI e = src[(int64_t)y * P.inner + x];
            tile[y * TX + x] = e;
            val[y * TX + x] = scaled_key<K>((uint32_t)e, y, si);
        }
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int g = warp % G, r0 = warp / G, rstep = nwarps / G;
    const int c = g * 32 + lane;
    if (c >= width) return;
    ColumnOut<K, FINAL> out;
    out.stride = P.inner;
    if (!FINAL) {
        using EO = typename EntryType<entry_bytes(K + 1)>::type;
        out.out = reinterpret_cast<EO*>(P.out) + slab * (int64_t)n * P.inner + i0 + c;
    } else {  // last pass: the slab is the image
        const int64_t v0 = i0 + c;
        out.dist = ep.dist ? ep.dist + slab * ep.V + v0 : nullptr;
        out.sq = nullptr;
        out.idx = ep.idx ? ep.idx + slab * ep.idx_planes * ep.V + v0 : nullptr;
        out.V = ep.V; out.ndim = ep.ndim;
        out.dist_only = ep.dist && !ep.idx;
        uint32_t rr = (uint32_t)v0;  // a position inside one image: below 2^31
#pragma unroll
        for (int q = 0; q < K; ++q) {
            const uint32_t nq = (uint32_t)ep.ext[q], hi = rr / nq;
            out.coord[q] = (int)(rr - hi * nq);
            rr = hi;
        }
#pragma unroll
        for (int q = 0; q <= K; ++q) out.axis[q] = ep.axis[q];
        out.init_index_planes(ep);
    }
    constexpr int R = 4;
    for (int y0 = r0 * R; y0 < n; y0 += rstep * R) {
        uint32_t best[R];
        scan_keys_group<TX, R, kScaledShift>(val + c, n, y0, best, (uint32_t)P.sk);
#pragma unroll
        for (int i = 0; i < R; ++i)
            if (y0 + i < n) emit_scaled<K, FINAL, EI>(out, tile + c, TX, y0 + i, best[i], P.inv_scale);
    }
}

}  // namespace tmedt
