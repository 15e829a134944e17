// Quad-per-lane kernels of the packed-entry path (extents up to 128, three or four processed axes, contiguous
// extent a multiple of 4, 16-byte aligned outputs): the same passes as edt_fast.cuh and edt_value.cuh,
//     g_k(x) = min_j [ g_{k-1}(x with x_k := j) + (w_k (x_k - j))^2 ]        (paper, Section 2.3.2)
// taken as exact bounded scans on integer keys, with a thread mapping chosen for instruction count:
//
//   * a lane owns four neighbouring voxels of ONE row of the axis (a "quad": four consecutive positions of the
//     contiguous index), so a candidate row is fetched with one 16-byte shared-memory load and serves four
//     voxels with the same addend (an immediate in the unrolled steps), and a quad's results leave in one or
//     two 16-byte stores;
//   * the key tile carries kLeanPad rows of "no site" keys above and below, so the first steps of every scan
//     run without bounds tests;
//   * nothing is decided per voxel that can be decided per block or per template instance.
//
// Keys: entries mode   (sum of squared offsets << 8) | row     (plane kernel: off^2 << 16 | row << 8 | off)
//       value mode     the squared distance so far, times the common scale in scaled-integer mode
// "No site" is 2^31 in both; every real key and every addend stays below it (checked by the planner).
#pragma once
#include "edt_debug.cuh"
#include "edt_fast.cuh"

namespace tmedt {

constexpr uint32_t kLeanNone = 0x80000000u;
constexpr int kLeanPad = 4;

struct LeanParams {
    const void* in;      // mask (plane kernel), entries or values of the earlier axes (column kernels)
    void* out;           // entries or values including this axis (unused by final kernels)
    int64_t inner;       // voxels between consecutive rows of the axis
    int n;               // extent of the axis
    int n0;              // plane kernel: extent of the contiguous axis
    int tiles_per_slab;  // column kernels: tiles of TX columns per (n x inner) slab
    uint32_t wk;         // integer weight of the axis: a row at distance d adds wk * d^2 (1 under unit sampling)
    uint32_t w0;         // plane kernel: integer weight of the contiguous axis
    float inv_scale;     // final value kernels: 1 / common scale (1 under unit sampling)
    int shift[4];        // final entry kernels: log2 of the extent of plane q, or -1 if it is no power of two
    int64_t in_elems;    // elements behind `in` and `out` (bounds checks of the debug build)
    int64_t out_elems;
    int64_t images;      // images behind the final outputs (bounds checks of the debug build)
    int reverse;         // column kernels: walk the blocks backwards (a pass between the plane pass and the last one:
                         // it starts with what the plane pass wrote last, still in L2, and ends with what the last pass,
                         // walking forwards, reads first)
    int dist16;          // value kernels, 16-bit input: the input holds first-axis distances (>= 0xC000: no site in the
                         // row) instead of squared values; they are squared while the tile is staged
};

// A key tile in shared memory: its first word and its size in words (bounds checks of the debug build).
struct LeanTile { const uint32_t* base; int words; };

__device__ __forceinline__ uint32_t lean_max4(const uint32_t (&b)[4]) { return max(max(b[0], b[1]), max(b[2], b[3])); }

__device__ __forceinline__ void lean_try_row(const LeanTile& T, const uint32_t* __restrict__ row, const uint32_t a,
                                             uint32_t (&b)[4]) {
    if (!TM_EDT_IN_RANGE(row - T.base, T.words - 3, 101)) return;
    const uint4 c = *reinterpret_cast<const uint4*>(row);
    b[0] = __viaddmin_u32(c.x, a, b[0]); b[1] = __viaddmin_u32(c.y, a, b[1]);
    b[2] = __viaddmin_u32(c.z, a, b[2]); b[3] = __viaddmin_u32(c.w, a, b[3]);
}

// Bounded scan of one quad.  own: the quad's keys inside the padded tile (row pitch PITCH words).
// Row distance d adds (wk d^2) << SH; a voxel is finished once that addend reaches its best key, so the work of a
// voxel grows with its distance to the background along the axis and never exceeds the extent.
template <int PITCH, int SH>
__device__ __forceinline__ void lean_scan(const LeanTile& T, const uint32_t* __restrict__ own, const int y, const int n,
                                          const uint32_t wk, uint32_t (&b)[4]) {
    b[0] = b[1] = b[2] = b[3] = kLeanNone;
    if (!TM_EDT_IN_RANGE(own - T.base, T.words - 3, 100)) return;
    {
        const uint4 v = *reinterpret_cast<const uint4*>(own);
        b[0] = v.x; b[1] = v.y; b[2] = v.z; b[3] = v.w;
    }
    uint32_t mx = lean_max4(b);
    if (mx < (1u << SH)) return;  // four background voxels
#pragma unroll
    for (int s = 1; s <= kLeanPad; ++s) {  // no bounds tests: the tile is padded
        if (s == 3 && ((wk * 9u) << SH) >= mx) return;
        const uint32_t a = (wk * (uint32_t)(s * s)) << SH;
        lean_try_row(T, own - s * PITCH, a, b);
        lean_try_row(T, own + s * PITCH, a, b);
        if (s == 2) mx = lean_max4(b);
    }
    mx = lean_max4(b);
    int d = kLeanPad + 1;
    uint32_t a = (wk * (uint32_t)(d * d)) << SH;
    if (a >= mx) return;
    const int up = y, dn = n - 1 - y, both = min(up, dn);
    const uint32_t* plo = own - d * PITCH;
    const uint32_t* phi = own + d * PITCH;
    // rows that exist on both sides, two distances per stop test
    for (; d + 1 <= both && a < mx; d += 2, plo -= 2 * PITCH, phi += 2 * PITCH) {
        const uint32_t a1 = (wk * (uint32_t)((d + 1) * (d + 1))) << SH;
        lean_try_row(T, plo, a, b);
        lean_try_row(T, phi, a, b);
        lean_try_row(T, plo - PITCH, a1, b);
        lean_try_row(T, phi + PITCH, a1, b);
        mx = lean_max4(b);
        a = (wk * (uint32_t)((d + 2) * (d + 2))) << SH;
    }
    // the rest: one distance at a time, the tile's ends tested
    for (; a < mx && (d <= up || d <= dn); ++d, plo -= PITCH, phi += PITCH) {
        if (d <= up) lean_try_row(T, plo, a, b);
        if (d <= dn) lean_try_row(T, phi, a, b);
        mx = lean_max4(b);
        a = (wk * (uint32_t)((d + 1) * (d + 1))) << SH;
    }
}

// "No site" rows above and below the tile.
template <int PITCH>
__device__ __forceinline__ void lean_fill_pad(uint32_t* __restrict__ kt, const int n) {
    constexpr int QPR = PITCH / 4;
    for (int t = threadIdx.x; t < 2 * kLeanPad * QPR; t += blockDim.x) {
        const int r = t / QPR, q = t - r * QPR;
        const int row = r < kLeanPad ? r : n + r;
        if (!TM_EDT_IN_RANGE(row * PITCH + 4 * q, (n + 2 * kLeanPad) * PITCH - 3, 102)) continue;
        *reinterpret_cast<uint4*>(kt + row * PITCH + 4 * q) = make_uint4(kLeanNone, kLeanNone, kLeanNone, kLeanNone);
    }
}

// ---------------------------------------------------------------------------------------------
// First-axis pass of one row into the key tile: one warp per row, four voxels per lane (one 32-bit load of the mask).
// Zero bytes are found with a carry-free byte test, the nearest lanes holding a zero on either side with one ballot
// and clz / ffs, their zero positions with two shuffles; the lane's four voxels are finished in registers.
//   ENT   key = off^2 << 16 | row << 8 | (off & 0xff)   (off = signed offset to the nearest zero of the row)
//   !ENT  key = w0 * off^2
// Returns the AND of the lane's four keys (all ones for lanes beyond the row): bit 31 stays set only if all are "no site".
// ---------------------------------------------------------------------------------------------
template <bool ENT>
__device__ __forceinline__ uint32_t lean_first_axis(const uint32_t v, const int n0, const int y, const uint32_t w0,
                                                uint32_t* __restrict__ krow, const int krow_words, const int lane) {
    const bool act = 4 * lane < n0;
    const uint32_t m = ~(((v & 0x7f7f7f7fu) + 0x7f7f7f7fu) | v) & 0x80808080u;  // 0x80 in every zero byte
    const unsigned any = __ballot_sync(0xffffffffu, m != 0u);  // lanes beyond the row hold foreground: m == 0
    uint4 keys;
    if (any == 0u) {  // no background in this row
        keys = make_uint4(kLeanNone, kLeanNone, kLeanNone, kLeanNone);
    } else if (__all_sync(0xffffffffu, m == 0x80808080u || !act)) {  // nothing but background
        const uint32_t k0 = ENT ? (uint32_t)y << 8 : 0u;
        keys = make_uint4(k0, k0, k0, k0);
    } else {
        // every lane of the warp stays in the shuffles; only the store is guarded
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
            kk[b] = ENT ? (((uint32_t)(a * a) << 16) | ((uint32_t)y << 8) | ((uint32_t)off & 0xffu)) : w0 * (uint32_t)(a * a);
        }
        keys = make_uint4(kk[0], kk[1], kk[2], kk[3]);
    }
    if (act && TM_EDT_IN_RANGE(4 * lane, krow_words - 3, 111)) *reinterpret_cast<uint4*>(krow + 4 * lane) = keys;
    return act ? (keys.x & keys.y & keys.z & keys.w) : 0xffffffffu;
}

// ---------------------------------------------------------------------------------------------
// First and second axis of one (n1 x n0) plane per block.
//   VT == uint8_t   entries: writes 2-byte entries (first-axis offset, second-axis offset)
//   VT == uint16_t  values:  writes the squared distance so far (all ones = no site)
//   VT == uint32_t  values:  writes the (scaled) squared distance so far (2^31 = no site)
// ---------------------------------------------------------------------------------------------
//   NW  warps per block: 8, or 16 where more resident warps are needed to cover the latencies of long scans
template <int VS, typename VT, int NW = 8>
__global__ void __launch_bounds__(32 * NW, 3) lean_plane_kernel(const __grid_constant__ LeanParams P) {
    constexpr bool ENT = sizeof(VT) == 1;
    constexpr int SH = ENT ? 16 : 0;
    extern __shared__ __align__(16) uint8_t sm_lean_p[];
    const int n0 = P.n0, n1 = P.n;
    uint32_t* kt = reinterpret_cast<uint32_t*>(sm_lean_p);      // [n1 + 2 kLeanPad][VS]
    const int64_t plane = blockIdx.x;
    const uint8_t* src = reinterpret_cast<const uint8_t*>(P.in) + plane * (int64_t)n1 * n0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t wk = ENT ? 1u : P.wk;
    lean_fill_pad<VS>(kt, n1);
    uint32_t all = 0xffffffffu;  // AND of this thread's keys
    {
        constexpr int MAXR = 128 / NW;  // rows per warp
        uint32_t rowv[MAXR];
        const bool act = 4 * lane < n0;
#pragma unroll
        for (int i = 0; i < MAXR; ++i) {  // all loads of this warp's rows are issued before the first row is processed
            const int y = warp + i * NW;
            rowv[i] = (act && y < n1 && TM_EDT_IN_RANGE(plane * (int64_t)n1 * n0 + y * n0 + 4 * lane, P.in_elems - 3, 110))
                          ? *reinterpret_cast<const uint32_t*>(src + y * n0 + 4 * lane) : 0x01010101u;
        }
#pragma unroll
        for (int i = 0; i < MAXR; ++i) {
            const int y = warp + i * NW;
            if (y < n1) all &= lean_first_axis<ENT>(rowv[i], n0, y, P.w0, kt + (y + kLeanPad) * VS, (n1 + kLeanPad - y) * VS, lane);
        }
    }
    // barrier; a plane without any background voxel needs no scan (every result is "no site")
    const int any_site = __syncthreads_or((all & kLeanNone) == 0u);
    // a warp takes patches of 4 rows x 32 columns (8 quads per row): neighbouring voxels have similar scan lengths
    constexpr int CG = VS / 32;
    const int r = lane >> 3, q4 = 4 * (lane & 7);
    const int64_t base0 = plane * (int64_t)n1 * n0;
    const int patches = ((n1 + 3) >> 2) * CG;
    const LeanTile T = {kt, (n1 + 2 * kLeanPad) * VS};
    for (int t = warp; t < patches; t += NW) {
        const int y = 4 * (t / CG) + r, c4 = 32 * (t % CG) + q4;
        if (y >= n1 || c4 >= n0) continue;
        uint32_t b[4];
        if (any_site) lean_scan<VS, SH>(T, kt + (y + kLeanPad) * VS + c4, y, n1, wk, b);
        else b[0] = b[1] = b[2] = b[3] = kLeanNone;
        const int64_t p = base0 + (int64_t)y * n0 + c4;
        if (!TM_EDT_IN_RANGE(p, P.out_elems - 3, 112)) continue;
        if (ENT) {
            uint32_t e[4];
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const uint32_t j = (b[v] >> 8) & 0xffu;
                e[v] = b[v] >= kLeanNone ? 0x80u : ((b[v] & 0xffu) | (((j - (uint32_t)y) & 0xffu) << 8));
            }
            *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(P.out) + p) = make_uint2(e[0] | (e[1] << 16), e[2] | (e[3] << 16));
        } else if (sizeof(VT) == 2) {
#pragma unroll
            for (int v = 0; v < 4; ++v) b[v] = min(b[v], 0xffffu);
            *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(P.out) + p) = make_uint2(b[0] | (b[1] << 16), b[2] | (b[3] << 16));
        } else {
            *reinterpret_cast<uint4*>(reinterpret_cast<uint32_t*>(P.out) + p) = make_uint4(b[0], b[1], b[2], b[3]);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// One further axis on entries (unit sampling, index output requested).  K earlier axes, K = 2 or 3.
//   FINAL == false  (K == 2)  writes 4-byte entries
//   FINAL == true             writes float32 distances and / or int64 squared distances, and the index planes
//                             (every spatial axis is a processed axis; FLAT: one linear index per voxel instead)
// ---------------------------------------------------------------------------------------------
// Four zero-extended 32-bit values as four int64: one 256-bit streaming store (p 32-byte aligned).
__device__ __forceinline__ void lean_store_4xi64(int64_t* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    const uint32_t z = 0u;
    asm volatile("st.global.cs.v8.b32 [%0], {%1, %5, %2, %5, %3, %5, %4, %5};"
                 :: "l"(p), "r"(a), "r"(b), "r"(c), "r"(d), "r"(z) : "memory");
}

// The same int64 (given as its two halves) four times: one 256-bit streaming store (p 32-byte aligned).
__device__ __forceinline__ void lean_store_4xi64_same(int64_t* p, uint32_t lo, uint32_t hi) {
    asm volatile("st.global.cs.v8.b32 [%0], {%1, %2, %1, %2, %1, %2, %1, %2};" :: "l"(p), "r"(lo), "r"(hi) : "memory");
}

__device__ __forceinline__ int lean_sext_byte(uint32_t e, int q) {
    // byte q of e, sign-extended: one byte-permute (bit 3 of a selector nibble replicates the sign of the byte)
    const uint32_t sel = (uint32_t)q | ((8u | (uint32_t)q) << 4) | ((8u | (uint32_t)q) << 8) | ((8u | (uint32_t)q) << 12);
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(e), "r"(0u), "r"(sel));
    return (int)r;
}

// Final outputs of one quad (index output requested, every spatial axis processed): b = the quad's final keys
// (squared distance << 8 | site row), e = the entries of the four sites along the K earlier axes, cq = the quad's own
// coordinates along those axes (plane 0 is the contiguous one: voxel v sits at cq[0] + v), p = its position inside
// the image, ip[q] = index plane of processed axis q.
template <int K>
__device__ __forceinline__ void lean_emit_final(const uint32_t (&b)[4], const uint32_t (&e)[4], const int (&cq)[K],
                                                float* __restrict__ dist, int64_t* __restrict__ sq,
                                                int64_t* const (&ip)[K + 1], const uint32_t p) {
    uint32_t j[4];
#pragma unroll
    for (int v = 0; v < 4; ++v) j[v] = b[v] & 0xffu;
    if (((b[0] | b[1] | b[2] | b[3]) & kLeanNone) == 0u) {
        if (dist) {
            float4 d;
            d.x = fast_sqrt(small_int_to_float((int)(b[0] >> 8))); d.y = fast_sqrt(small_int_to_float((int)(b[1] >> 8)));
            d.z = fast_sqrt(small_int_to_float((int)(b[2] >> 8))); d.w = fast_sqrt(small_int_to_float((int)(b[3] >> 8)));
            __stcs(reinterpret_cast<float4*>(dist + p), d);
        }
        if (sq) lean_store_4xi64(sq + p, b[0] >> 8, b[1] >> 8, b[2] >> 8, b[3] >> 8);
#pragma unroll
        for (int q = 0; q < K; ++q) {
            uint32_t s[4];
#pragma unroll
            for (int v = 0; v < 4; ++v) s[v] = (uint32_t)(cq[q] + (q == 0 ? v : 0) + lean_sext_byte(e[v], q));
            lean_store_4xi64(ip[q] + p, s[0], s[1], s[2], s[3]);
        }
        lean_store_4xi64(ip[K] + p, j[0], j[1], j[2], j[3]);
    } else if ((b[0] & b[1] & b[2] & b[3] & kLeanNone) != 0u) {  // an image without background: +inf, INT64_MAX, -1
        if (dist) __stcs(reinterpret_cast<float4*>(dist + p), make_float4(TMEDT_INF, TMEDT_INF, TMEDT_INF, TMEDT_INF));
        if (sq) lean_store_4xi64_same(sq + p, 0xffffffffu, 0x7fffffffu);
#pragma unroll
        for (int q = 0; q <= K; ++q) lean_store_4xi64_same(ip[q] + p, 0xffffffffu, 0xffffffffu);
    } else {  // cannot happen inside one image (all its voxels have a site or none has); kept voxel by voxel
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const bool none = b[v] >= kLeanNone;
            if (dist) dist[p + v] = none ? TMEDT_INF : fast_sqrt(small_int_to_float((int)(b[v] >> 8)));
            if (sq) sq[p + v] = none ? INT64_MAX : (int64_t)(b[v] >> 8);
#pragma unroll
            for (int q = 0; q < K; ++q)
                ip[q][p + v] = none ? (int64_t)-1 : (int64_t)(cq[q] + (q == 0 ? v : 0) + lean_sext_byte(e[v], q));
            ip[K][p + v] = none ? (int64_t)-1 : (int64_t)j[v];
        }
    }
}

// The same with one linear index per voxel (the site's row-major position inside its image) instead of coordinate
// planes: the quad's own position p + v, moved by the entry's offsets along the K earlier planes (strides ps[q]) and by
// the site row along this axis (own row y, stride inner).
template <int K>
__device__ __forceinline__ void lean_emit_flat(const uint32_t (&b)[4], const uint32_t (&e)[4], float* __restrict__ dist,
                                               int64_t* __restrict__ sq, int64_t* __restrict__ lin, const uint32_t p,
                                               const int y, const int inner, const int (&ps)[K]) {
    const uint32_t any = b[0] | b[1] | b[2] | b[3], every = b[0] & b[1] & b[2] & b[3];
    if ((any & kLeanNone) == 0u) {
        if (dist) {
            float4 d;
            d.x = fast_sqrt(small_int_to_float((int)(b[0] >> 8))); d.y = fast_sqrt(small_int_to_float((int)(b[1] >> 8)));
            d.z = fast_sqrt(small_int_to_float((int)(b[2] >> 8))); d.w = fast_sqrt(small_int_to_float((int)(b[3] >> 8)));
            __stcs(reinterpret_cast<float4*>(dist + p), d);
        }
        if (sq) lean_store_4xi64(sq + p, b[0] >> 8, b[1] >> 8, b[2] >> 8, b[3] >> 8);
        uint32_t s[4];
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            int at = (int)p + v + ((int)(b[v] & 0xffu) - y) * inner;
#pragma unroll
            for (int q = 0; q < K; ++q) at += lean_sext_byte(e[v], q) * ps[q];
            s[v] = (uint32_t)at;
        }
        lean_store_4xi64(lin + p, s[0], s[1], s[2], s[3]);
    } else if ((every & kLeanNone) != 0u) {  // an image without background: +inf, INT64_MAX, -1
        if (dist) __stcs(reinterpret_cast<float4*>(dist + p), make_float4(TMEDT_INF, TMEDT_INF, TMEDT_INF, TMEDT_INF));
        if (sq) lean_store_4xi64_same(sq + p, 0xffffffffu, 0x7fffffffu);
        lean_store_4xi64_same(lin + p, 0xffffffffu, 0xffffffffu);
    } else {  // cannot happen inside one image; kept voxel by voxel
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const bool none = b[v] >= kLeanNone;
            if (dist) dist[p + v] = none ? TMEDT_INF : fast_sqrt(small_int_to_float((int)(b[v] >> 8)));
            if (sq) sq[p + v] = none ? INT64_MAX : (int64_t)(b[v] >> 8);
            int at = (int)p + v + ((int)(b[v] & 0xffu) - y) * inner;
#pragma unroll
            for (int q = 0; q < K; ++q) at += lean_sext_byte(e[v], q) * ps[q];
            lin[p + v] = none ? (int64_t)-1 : (int64_t)at;
        }
    }
}

// Own coordinates along the K earlier planes of position v0 (plane 0 fastest).
template <int K>
__device__ __forceinline__ void lean_decode(uint32_t v0, const LeanParams& P, const EpilogueParams& ep, int (&cq)[K]) {
#pragma unroll
    for (int q = 0; q < K; ++q) {
        if (P.shift[q] >= 0) {
            cq[q] = (int)(v0 & (((uint32_t)1 << P.shift[q]) - 1u));
            v0 >>= P.shift[q];
        } else {
            const uint32_t nq = (uint32_t)ep.ext[q], hi = v0 / nq;
            cq[q] = (int)(v0 - hi * nq);
            v0 = hi;
        }
    }
}

template <int K, bool FINAL, int TX, bool FLAT = false>
__global__ void __launch_bounds__(256, FINAL ? 6 : 8) lean_column_kernel(const __grid_constant__ LeanParams P,
                                                                         const __grid_constant__ EpilogueParams ep) {
    using EI = typename EntryType<entry_bytes(K)>::type;
    constexpr int LPR = TX / 4, CG = TX / 32, NW = 8;
    extern __shared__ __align__(16) uint8_t sm_lean_c[];
    const int n = P.n;
    uint32_t* kt = reinterpret_cast<uint32_t*>(sm_lean_c);                                  // [n + 2 kLeanPad][TX]
    EI* et = reinterpret_cast<EI*>(sm_lean_c + (size_t)(n + 2 * kLeanPad) * TX * 4);        // [n][TX]
    const unsigned bid = P.reverse ? gridDim.x - 1 - blockIdx.x : blockIdx.x;
    const int64_t slab = bid / P.tiles_per_slab;
    const int64_t i0 = (int64_t)(bid - slab * P.tiles_per_slab) * TX;
    const int width = (int)min((int64_t)TX, P.inner - i0);
    const EI* src = reinterpret_cast<const EI*>(P.in) + slab * (int64_t)n * P.inner + i0;
    lean_fill_pad<TX>(kt, n);
    uint32_t all = 0xffffffffu;  // AND of this thread's keys
#pragma unroll 4
    for (int t = threadIdx.x; t < n * LPR; t += 256) {
        const int y = t / LPR, q4 = 4 * (t % LPR);
        if (q4 >= width) continue;
        const EI* g = src + (int64_t)y * P.inner + q4;
        if (!TM_EDT_IN_RANGE(g - reinterpret_cast<const EI*>(P.in), P.in_elems - 3, 120)) continue;
        uint32_t e[4];
        if (sizeof(EI) == 2) {
            const uint2 w = *reinterpret_cast<const uint2*>(g);
            *reinterpret_cast<uint2*>(et + y * TX + q4) = w;
            e[0] = w.x & 0xffffu; e[1] = w.x >> 16; e[2] = w.y & 0xffffu; e[3] = w.y >> 16;
        } else {
            const uint4 w = *reinterpret_cast<const uint4*>(g);
            *reinterpret_cast<uint4*>(et + y * TX + q4) = w;
            e[0] = w.x; e[1] = w.y; e[2] = w.z; e[3] = w.w;
        }
        uint32_t k[4];
#pragma unroll
        for (int v = 0; v < 4; ++v)
            k[v] = e[v] == 0x80u ? kLeanNone : (((uint32_t)__dp4a((int)e[v], (int)e[v], 0) << 8) | (uint32_t)y);
        *reinterpret_cast<uint4*>(kt + (y + kLeanPad) * TX + q4) = make_uint4(k[0], k[1], k[2], k[3]);
        all &= k[0] & k[1] & k[2] & k[3];
    }
    // barrier; a tile without any site (an image without background) needs no scan
    const int any_site = __syncthreads_or((all & kLeanNone) == 0u);
    // a warp takes patches of 4 rows x 32 columns (8 quads per row), always in the same 32 columns
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c4 = 32 * (warp % CG) + 4 * (lane & 7);
    const int yfirst = 4 * (warp / CG) + (lane >> 3);
    constexpr int YSTEP = 4 * (NW / CG);
    if (c4 >= width) return;
    const uint32_t v0 = (uint32_t)(i0 + c4);  // the quad's position among the earlier planes (plane 0 fastest)
    const LeanTile T = {kt, (n + 2 * kLeanPad) * TX};
    if (!FINAL) {
        uint32_t* out = reinterpret_cast<uint32_t*>(P.out) + slab * (int64_t)n * P.inner + v0;
        for (int y = yfirst; y < n; y += YSTEP) {
            uint32_t b[4], o[4];
            if (any_site) lean_scan<TX, 8>(T, kt + (y + kLeanPad) * TX + c4, y, n, 1u, b);
            else b[0] = b[1] = b[2] = b[3] = kLeanNone;
            if (!TM_EDT_IN_RANGE(slab * (int64_t)n * P.inner + v0 + (int64_t)y * P.inner, P.out_elems - 3, 121)) continue;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const uint32_t j = TM_EDT_IN_RANGE(b[v] & 0xffu, n, 122) ? (b[v] & 0xffu) : 0u;
                const uint32_t e = (uint32_t)et[j * TX + c4 + v];
                o[v] = b[v] >= kLeanNone ? 0x80u : (e | (((j - (uint32_t)y) & 0xffu) << (8 * K)));
            }
            *reinterpret_cast<uint4*>(out + (int64_t)y * P.inner) = make_uint4(o[0], o[1], o[2], o[3]);
        }
        return;
    }
    float* const dist = ep.dist ? ep.dist + slab * ep.V : nullptr;
    int64_t* const sq = ep.sq ? ep.sq + slab * ep.V : nullptr;
    if (FLAT) {  // one linear index per voxel
        int ps[K];
#pragma unroll
        for (int q = 0; q < K; ++q) ps[q] = (int)ep.pstride[q];
        int64_t* const lin = ep.idx + slab * ep.V;
        for (int y = yfirst; y < n; y += YSTEP) {
            uint32_t b[4], e[4];
            if (any_site) lean_scan<TX, 8>(T, kt + (y + kLeanPad) * TX + c4, y, n, 1u, b);
            else b[0] = b[1] = b[2] = b[3] = kLeanNone;
#pragma unroll
            for (int v = 0; v < 4; ++v) e[v] = (uint32_t)et[(TM_EDT_IN_RANGE(b[v] & 0xffu, n, 126) ? (b[v] & 0xffu) : 0u) * TX + c4 + v];
            const uint32_t p = (uint32_t)y * (uint32_t)P.inner + v0;  // inside one image: below 2^31
            if (TM_EDT_IN_RANGE(p, ep.V - 3, 127) && TM_EDT_IN_RANGE(slab, P.images, 128))
                lean_emit_flat<K>(b, e, dist, sq, lin, p, y, (int)P.inner, ps);
        }
        return;
    }
    int cq[K];
    lean_decode<K>(v0, P, ep, cq);
    int64_t* ip[K + 1];
#pragma unroll
    for (int q = 0; q <= K; ++q) ip[q] = ep.idx + (slab * ep.ndim + ep.axis[q]) * ep.V;
    for (int y = yfirst; y < n; y += YSTEP) {
        uint32_t b[4], e[4];
        if (any_site) lean_scan<TX, 8>(T, kt + (y + kLeanPad) * TX + c4, y, n, 1u, b);
        else b[0] = b[1] = b[2] = b[3] = kLeanNone;
#pragma unroll
        for (int v = 0; v < 4; ++v) e[v] = (uint32_t)et[(TM_EDT_IN_RANGE(b[v] & 0xffu, n, 123) ? (b[v] & 0xffu) : 0u) * TX + c4 + v];
        const uint32_t p = (uint32_t)y * (uint32_t)P.inner + v0;  // inside one image: below 2^31
        if (TM_EDT_IN_RANGE(p, ep.V - 3, 124) && TM_EDT_IN_RANGE(slab, P.images, 125))
            lean_emit_final<K>(b, e, cq, dist, sq, ip, p);
    }
}

// ---------------------------------------------------------------------------------------------
// One further axis on carried values (no index output): the key is the value itself.
//   VT  uint16_t (all ones = no site) or uint32_t (2^31 = no site)
//   FINAL == false  writes the new value;  FINAL == true  writes float32 distances and / or int64 squared distances
// ---------------------------------------------------------------------------------------------
template <bool FINAL, typename VT, int TX, int NW = 8>
__global__ void __launch_bounds__(32 * NW) lean_value_kernel(const __grid_constant__ LeanParams P,
                                                            const __grid_constant__ EpilogueParams ep) {
    // tiles of 4, 8 or 16 columns (axes beyond 1024 rows): a warp's patch is 32, 16 or 8 rows of the whole tile width
    constexpr int LPR = TX / 4, CG = TX >= 32 ? TX / 32 : 1, RPW = TX >= 32 ? 4 : 128 / TX;
    extern __shared__ __align__(16) uint8_t sm_lean_v[];
    const int n = P.n;
    uint32_t* kt = reinterpret_cast<uint32_t*>(sm_lean_v);  // [n + 2 kLeanPad][TX]
    const int64_t slab = blockIdx.x / P.tiles_per_slab;
    const int64_t i0 = (int64_t)(blockIdx.x - slab * P.tiles_per_slab) * TX;
    const int width = (int)min((int64_t)TX, P.inner - i0);
    const VT* src = reinterpret_cast<const VT*>(P.in) + slab * (int64_t)n * P.inner + i0;
    lean_fill_pad<TX>(kt, n);
    uint32_t all = 0xffffffffu;  // AND of this thread's keys
#pragma unroll 4
    for (int t = threadIdx.x; t < n * LPR; t += 32 * NW) {
        const int y = t / LPR, q4 = 4 * (t % LPR);
        if (q4 >= width) continue;
        const VT* g = src + (int64_t)y * P.inner + q4;
        if (!TM_EDT_IN_RANGE(g - reinterpret_cast<const VT*>(P.in), P.in_elems - 3, 130)) continue;
        uint4 k;
        if (sizeof(VT) == 2) {
            const uint2 w = *reinterpret_cast<const uint2*>(g);
            k = make_uint4(w.x & 0xffffu, w.x >> 16, w.y & 0xffffu, w.y >> 16);
            if (P.dist16) {
                k.x = k.x >= 0xC000u ? kLeanNone : k.x * k.x * P.w0;  // (w0: 1, or the integer weight of scaled sampling)
                k.y = k.y >= 0xC000u ? kLeanNone : k.y * k.y * P.w0;
                k.z = k.z >= 0xC000u ? kLeanNone : k.z * k.z * P.w0;
                k.w = k.w >= 0xC000u ? kLeanNone : k.w * k.w * P.w0;
            } else {
                if (k.x == 0xffffu) k.x = kLeanNone;
                if (k.y == 0xffffu) k.y = kLeanNone;
                if (k.z == 0xffffu) k.z = kLeanNone;
                if (k.w == 0xffffu) k.w = kLeanNone;
            }
        } else {
            k = *reinterpret_cast<const uint4*>(g);
        }
        *reinterpret_cast<uint4*>(kt + (y + kLeanPad) * TX + q4) = k;
        all &= k.x & k.y & k.z & k.w;
    }
    const int any_site = __syncthreads_or((all & kLeanNone) == 0u);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c4 = TX >= 32 ? 32 * (warp % CG) + 4 * (lane & 7) : 4 * (lane % LPR);
    const int yfirst = TX >= 32 ? 4 * (warp / CG) + (lane >> 3) : RPW * warp + lane / LPR;
    constexpr int YSTEP = RPW * (NW / CG);
    if (c4 >= width) return;
    const int64_t col = slab * (int64_t)n * P.inner + i0 + c4;  // FINAL: the slab is the image
    const LeanTile T = {kt, (n + 2 * kLeanPad) * TX};
    for (int y = yfirst; y < n; y += YSTEP) {
        uint32_t b[4];
        if (any_site) lean_scan<TX, 0>(T, kt + (y + kLeanPad) * TX + c4, y, n, P.wk, b);
        else b[0] = b[1] = b[2] = b[3] = kLeanNone;
        const int64_t p = col + (int64_t)y * P.inner;
        if (!TM_EDT_IN_RANGE(p, (FINAL ? P.images * ep.V : P.out_elems) - 3, 131)) continue;
        if (!FINAL) {
            if (sizeof(VT) == 2 && !P.dist16) {  // (16-bit row distances in: 32-bit values out)
#pragma unroll
                for (int v = 0; v < 4; ++v) b[v] = min(b[v], 0xffffu);
                *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(P.out) + p) = make_uint2(b[0] | (b[1] << 16), b[2] | (b[3] << 16));
            } else {
                *reinterpret_cast<uint4*>(reinterpret_cast<uint32_t*>(P.out) + p) = make_uint4(b[0], b[1], b[2], b[3]);
            }
            continue;
        }
        const uint32_t all = b[0] | b[1] | b[2] | b[3];
        if (ep.dist) {
            float4 d = make_float4(0.f, 0.f, 0.f, 0.f);
            if (all != 0u) {
                float f[4];
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    // exact integer below 2^24 -> float32: two full-rate operations below 2^23, a conversion otherwise
                    const float x = all < (1u << 23) ? small_int_to_float((int)b[v]) : __uint2float_rn(b[v]);
                    f[v] = b[v] >= kLeanNone ? TMEDT_INF : fast_sqrt(x * P.inv_scale);
                }
                d = make_float4(f[0], f[1], f[2], f[3]);
            }
            __stcs(reinterpret_cast<float4*>(ep.dist + p), d);
        }
        if (ep.sq) {  // unit sampling only
            if ((all & kLeanNone) == 0u) {
                lean_store_4xi64(ep.sq + p, b[0], b[1], b[2], b[3]);
            } else {
#pragma unroll
                for (int v = 0; v < 4; ++v) ep.sq[p + v] = b[v] >= kLeanNone ? INT64_MAX : (int64_t)b[v];
            }
        }
    }
}

}  // namespace tmedt
