// Extents beyond the 128 of the packed 8-bit entries, two to four processed axes, extents up to 1024.
// Kernels:
//   row_keys_kernel     first-axis pass, one warp per row, 16 or 32 voxels per lane (128-bit loads; rows that
//                       are not 16-byte aligned use long_row_any_kernel of edt_long.cuh instead).
//                       Writes, per voxel, the scan value and the signed 16-bit offset to the nearest zero of
//                       the row.  Unit sampling: the key (off^2 << SH) | row (32 bit; SH = 9 row bits for
//                       extents up to 512, 10 up to 1024), as long as every key stays below 2^31 (two axes up
//                       to 1024, three up to about 830).  Otherwise: the float32 height w^2 off^2.
//   wide_axis_kernel    every further axis: a block stages the values of an (n x 32) strip in shared memory and
//                       runs the bounded scan on it (grouped, edt_fast.cuh, for keys).  A middle pass writes
//                       the value of the next pass and the site's offsets (16 bits per axis); the last pass
//                       writes the outputs and fetches the chosen site's offsets only when indices are requested.
// Same mathematics as the fast path: g_k(x) = min_j [ g_{k-1}(x with x_k := j) + (w_k (x_k - j))^2 ], exact in
// integers under unit sampling.
#pragma once
#include "edt_fast.cuh"

namespace tmedt {


struct WideParams {
    const uint8_t* in;   // (images, n1, n0)
    uint32_t* keys;      // (images, n1, n0)
    int16_t* offs;       // (images, n1, n0), or nullptr when no index output is requested
    int64_t rows;        // images * n1
    int n0, n1;
    float w2x;           // squared sampling of the contiguous axis (float-height variant)
    uint32_t w0i;        // its integer weight (plain integer values, SH == 0 or the long-line path; 1 under unit sampling)
};

// SH > 0: integer keys (off^2 << SH | row).  SH == 0: the plain integer off^2 (no site is needed afterwards: no index
// output).  SH < 0: float32 heights w^2 off^2 for general sampling (+inf = no site).
template <int VPL, int SH>  // voxels per lane (16 or 32), row bits of the key
__global__ void __launch_bounds__(256) row_keys_kernel(const __grid_constant__ WideParams P) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= P.rows) return;  // the whole warp leaves together
    const int n0 = P.n0;
    const int y = (int)(row % P.n1);
    const uint8_t* src = P.in + row * n0;
    constexpr int CH = VPL / 16;  // 16-byte chunks per lane
    uint32_t zb = 0u;             // bit b set: voxel b of this lane is zero
#pragma unroll
    for (int c = 0; c < CH; ++c) {
        uint4 v = make_uint4(0x01010101u, 0x01010101u, 0x01010101u, 0x01010101u);
        if (VPL * lane + 16 * c < n0) v = *reinterpret_cast<const uint4*>(src + VPL * lane + 16 * c);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t m = ~(((w[i] & 0x7f7f7f7fu) + 0x7f7f7f7fu) | w[i]) & 0x80808080u;
            // gather the four flag bits (bits 7, 15, 23, 31) into bits 0..3
            zb |= ((((m >> 7) * 0x00204081u) >> 21) & 0xfu) << (16 * c + 4 * i);
        }
    }
    const unsigned any = __ballot_sync(0xffffffffu, zb != 0u);
    uint32_t keys[VPL];
    int16_t offs[VPL];
    if (any == 0u) {
#pragma unroll
        for (int b = 0; b < VPL; ++b) { keys[b] = SH < 0 ? 0x7f800000u : kNoneKey16; offs[b] = (int16_t)-32768; }
    } else {
        const int lzin = zb ? 31 - __clz(zb) : 0;
        const int fzin = zb ? __ffs(zb) - 1 : 0;
        const unsigned ml = any & ((1u << lane) - 1u);
        const unsigned mr = lane < 31 ? any >> (lane + 1) : 0u;
        const int Ll = ml ? 31 - __clz(ml) : 0;
        const int Lr = mr ? lane + __ffs(mr) : 0;
        const int lz_l = __shfl_sync(0xffffffffu, lzin, Ll);
        const int fz_r = __shfl_sync(0xffffffffu, fzin, Lr);
        const int x0 = VPL * lane;
        int dl[VPL];
        int cur = ml ? VPL * Ll + lz_l : -4096;
#pragma unroll
        for (int b = 0; b < VPL; ++b) {
            if ((zb >> b) & 1u) cur = x0 + b;
            dl[b] = x0 + b - cur;
        }
        cur = mr ? VPL * Lr + fz_r : 8192;
#pragma unroll
        for (int b = VPL - 1; b >= 0; --b) {
            if ((zb >> b) & 1u) cur = x0 + b;
            const int dr = cur - (x0 + b);
            const int a = min(dl[b], dr);
            offs[b] = (int16_t)(dl[b] <= dr ? -a : a);
            keys[b] = SH < 0 ? __float_as_uint(P.w2x * (float)(a * a)) : (SH == 0 ? (uint32_t)(a * a) * P.w0i : (((uint32_t)(a * a) << (SH < 0 ? 0 : SH)) | (uint32_t)y));
        }
    }
#pragma unroll
    for (int c = 0; c < CH; ++c) {
        if (VPL * lane + 16 * c < n0) {
            uint4* kdst = reinterpret_cast<uint4*>(P.keys + row * n0 + VPL * lane + 16 * c);
#pragma unroll
            for (int i = 0; i < 4; ++i)
                kdst[i] = make_uint4(keys[16 * c + 4 * i], keys[16 * c + 4 * i + 1], keys[16 * c + 4 * i + 2],
                                     keys[16 * c + 4 * i + 3]);
            if (P.offs) {  // offsets are carried only when the index output is requested
                uint32_t pk[8];
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    pk[i] = (uint32_t)(uint16_t)offs[16 * c + 2 * i] | ((uint32_t)(uint16_t)offs[16 * c + 2 * i + 1] << 16);
                uint4* odst = reinterpret_cast<uint4*>(P.offs + row * n0 + VPL * lane + 16 * c);
                odst[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                odst[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
            }
        }
    }
}

// One further axis of the wide path.  The array is viewed as (outer, n, inner); a block takes one slab and
// a strip of 32 consecutive `inner` positions, stages the keys of its n rows in shared memory and runs the
// grouped bounded scan.  K = number of 16-bit offsets every voxel carries so far (1, 2 or 3).
//   FINAL == false  writes the key of the next pass (value << SH | index of the slab along the next axis)
//                   and K + 1 offsets per voxel (the chosen site's offsets, fetched from global memory, plus
//                   the offset along this axis);
//   FINAL == true   writes distances, squared distances and index planes (the slab is the image).
struct WideAxisParams {
    const uint32_t* keys_in;   // (outer, n, inner)
    const int16_t* offs_in;    // (outer, n, inner, K)  -- three offsets are stored as four (8 bytes per voxel)
    uint32_t* keys_out;        // (outer, n, inner), unused when FINAL
    int16_t* offs_out;         // (outer, n, inner, K + 1), unused when FINAL
    int64_t outer, inner;
    int n;
    int next_n;                // extent of the next axis (non-final)
    int n0;                    // extent of the contiguous axis (to split an inner position into coordinates)
    int n1;                    // extent of the second axis (fourth-axis pass only)
    float w2;                  // squared sampling of this axis (float-height variant)
    int row_parts;             // blocks that share one strip, each taking a contiguous range of its rows
};

// Bounded scan of one voxel on float32 heights (general sampling): returns the best value and the distance bd
// (0 = own row) at which it was found; the caller resolves the side.
template <int VS>
__device__ __forceinline__ float scan_heights_plain(const uint32_t* __restrict__ col, int n, int y, float w2, int& bd) {
    float best = __uint_as_float(col[y * VS]);
    bd = 0;
    float fd = 1.0f;
    for (int d = 1; d < n; ++d, fd += 1.0f) {
        const float add = w2 * fd * fd;
        if (add >= best) break;
        if (y - d < 0 && y + d >= n) break;
        const float lo = y - d >= 0 ? __uint_as_float(col[(y - d) * VS]) : TMEDT_INF;
        const float hi = y + d < n ? __uint_as_float(col[(y + d) * VS]) : TMEDT_INF;
        const float c = fminf(lo, hi) + add;
        if (c < best) { best = c; bd = d; }
    }
    return best;
}

// CW: columns of a strip (32, or 16 for long axes: smaller tiles, more blocks per SM, two row groups per warp)
template <int K, bool FINAL, int SH, int CW = 32>
__global__ void __launch_bounds__(512) wide_axis_kernel(const __grid_constant__ WideAxisParams P,
                                                        const __grid_constant__ EpilogueParams ep,
                                                        const int strips_per_slab) {
    extern __shared__ __align__(16) uint8_t sm_wide[];
    uint32_t* val = reinterpret_cast<uint32_t*>(sm_wide);  // [n][CW]
    const int n = P.n;
    const unsigned part = blockIdx.x % (unsigned)P.row_parts, sidx = blockIdx.x / (unsigned)P.row_parts;
    const int64_t slab = sidx / (unsigned)strips_per_slab;
    const int64_t c0 = (int64_t)(sidx - slab * strips_per_slab) * CW;
    const int64_t slab_base = slab * (int64_t)n * P.inner;
    const uint32_t* src = P.keys_in + slab_base + c0;
    // rows of this block (a multiple of R per part); every part stages the whole strip, a scan may reach any row
    const int rows_per_part = ((n + P.row_parts - 1) / P.row_parts + 3) & ~3;
    const int y_begin = (int)part * rows_per_part, y_end = min(n, y_begin + rows_per_part);
    // stage: CW / 4 threads copy one row of keys in 16-byte pieces when rows are 16-byte aligned, single keys otherwise
    const int width = (int)min((int64_t)CW, P.inner - c0);
    constexpr int TPR = CW / 4;
    if ((P.inner & 3) == 0) {
        for (int t = threadIdx.x; t < n * TPR; t += blockDim.x) {
            const int y = t / TPR, ch = t % TPR;
            if (4 * ch < width)
                *reinterpret_cast<uint4*>(val + y * CW + 4 * ch) = *reinterpret_cast<const uint4*>(src + (int64_t)y * P.inner + 4 * ch);
        }
    } else {
        for (int t = threadIdx.x; t < n * CW; t += blockDim.x) {
            const int y = t / CW, x = t % CW;
            if (x < width) val[y * CW + x] = src[(int64_t)y * P.inner + x];
        }
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    constexpr int GPW = 32 / CW;  // row groups a warp works on at a time
    const int lane = threadIdx.x & (CW - 1), sub = (threadIdx.x & 31) / CW;
    if (lane >= width) return;
    const int64_t c = c0 + lane;  // position along inner
    constexpr int R = 4;
    constexpr uint32_t kRowMask = SH < 0 ? 0u : (1u << (SH < 0 ? 0 : SH)) - 1u;
    const int64_t col_base = slab_base + c;  // voxel (row 0) of this column
    const uint32_t next_row = (FINAL || SH == 0) ? 0u : (uint32_t)(slab % P.next_n);  // SH == 0: plain values, no row bits
    // own coordinates along the earlier axes (final pass, index output): plane 0 = contiguous axis
    const int cx = (int)(c % P.n0);
    const int cyz = (int)(c / P.n0);
    const int cy = K == 3 ? cyz % P.n1 : cyz, cz = K == 3 ? cyz / P.n1 : 0;
    for (int y0 = y_begin + (warp * GPW + sub) * R; y0 < y_end; y0 += nwarps * GPW * R) {
        uint32_t best[R];
        int jrow[R];
        if (SH >= 0) {
            scan_keys_group<CW, R, (SH < 0 ? 9 : SH)>(val + lane, n, y0, best);
#pragma unroll
            for (int i = 0; i < R; ++i) jrow[i] = (int)(best[i] & kRowMask);
        } else {
#pragma unroll
            for (int i = 0; i < R; ++i) {
                const int y = y0 + i;
                best[i] = 0u; jrow[i] = y;
                if (y >= n) continue;
                int bd;
                best[i] = __float_as_uint(scan_heights_plain<CW>(val + lane, n, y, P.w2, bd));
                if (bd > 0) {
                    const float lo = y - bd >= 0 ? __uint_as_float(val[(y - bd) * CW + lane]) : TMEDT_INF;
                    const float hi = y + bd < n ? __uint_as_float(val[(y + bd) * CW + lane]) : TMEDT_INF;
                    jrow[i] = lo <= hi ? y - bd : y + bd;
                }
            }
        }
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int y = y0 + i;
            if (y >= n) break;
            const uint32_t b = best[i];
            const bool none = SH < 0 ? b == 0x7f800000u : b >= kNoneKey16;
            const int j = jrow[i];
            const int64_t p = col_base + (int64_t)y * P.inner;    // this voxel
            const int64_t pj = col_base + (int64_t)j * P.inner;   // the chosen site's voxel of this column
            if (!FINAL) {
                if (SH < 0) P.keys_out[p] = b;  // the height itself is the next pass's scan value
                else P.keys_out[p] = none ? kNoneKey16 : ((b & ~kRowMask) | next_row);
                if (!P.offs_out) {
                    // distances only: no offsets are carried
                } else if (K == 1) {
                    const uint32_t o0 = none ? 0x8000u : (uint32_t)(uint16_t)P.offs_in[pj];
                    reinterpret_cast<uint32_t*>(P.offs_out)[p] = o0 | ((uint32_t)(uint16_t)(int16_t)(j - y) << 16);
                } else if (K == 2) {
                    const uint32_t o01 = none ? 0x8000u : reinterpret_cast<const uint32_t*>(P.offs_in)[pj];
                    reinterpret_cast<uint2*>(P.offs_out)[p] = make_uint2(o01, (uint32_t)(uint16_t)(int16_t)(j - y));
                }
            } else {
                const int sq = SH < 0 ? 0 : (int)(b >> (SH < 0 ? 0 : SH));
                if (ep.dist)
                    ep.dist[p] = none ? TMEDT_INF
                                      : (SH < 0 ? __fsqrt_rn(__uint_as_float(b)) : __fsqrt_rn(small_int_to_float(sq)));
                if (ep.sq) ep.sq[p] = none ? INT64_MAX : (int64_t)sq;  // unit sampling only
                if (ep.idx) {
                    // processed axes in plane order: contiguous axis, (second axis,) this axis; others have extent 1
                    int site[4] = {0, 0, 0, 0};
                    if (!none) {
                        if (K == 1) {
                            site[0] = cx + (int)P.offs_in[pj];
                            site[1] = j;
                        } else if (K == 2) {
                            const uint32_t o = reinterpret_cast<const uint32_t*>(P.offs_in)[pj];
                            site[0] = cx + (int)(int16_t)(o & 0xffffu);
                            site[1] = cy + (int)(int16_t)(o >> 16);
                            site[2] = j;
                        } else {
                            const uint2 o = reinterpret_cast<const uint2*>(P.offs_in)[pj];
                            site[0] = cx + (int)(int16_t)(o.x & 0xffffu);
                            site[1] = cy + (int)(int16_t)(o.x >> 16);
                            site[2] = cz + (int)(int16_t)(o.y & 0xffffu);
                            site[3] = j;
                        }
                    }
                    const int64_t vox = p - slab_base;  // voxel index inside the image
                    if (ep.flat) {
                        int64_t f = 0;
#pragma unroll
                        for (int q = 0; q <= K; ++q) f += (int64_t)site[q] * ep.pstride[q];
                        ep.idx[slab * ep.V + vox] = none ? -1 : f;
                    } else
                    for (int a = 0; a < ep.ndim; ++a) {
                        int64_t v = 0;
#pragma unroll
                        for (int q = 0; q <= K; ++q)
                            if (a == ep.axis[q]) v = site[q];
                        ep.idx[(slab * ep.ndim + a) * ep.V + vox] = none ? -1 : v;
                    }
                }
            }
        }
    }
}

}  // namespace tmedt
