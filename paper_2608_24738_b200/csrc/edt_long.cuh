// Long lines: two or three processed axes with extents up to 8192 (beyond the 1024 rows a shared-memory
// strip of the wide path can hold).  Same mathematics as everywhere else,
//     g_k(x) = min_j [ g_{k-1}(x with x_k := j) + (w_k (x_k - j))^2 ]      (paper, Section 2.3.2)
// on plain 32-bit heights: exact unsigned integers under unit sampling (3 * 8191^2 < 2^28), float32
// otherwise.  Non-negative floats order like their bit patterns, so both kinds share the unsigned minimum;
// only the candidate's addition differs.  Kernels:
//   long_row_kernel    first-axis pass, one warp per row, 1024 voxels (32 per lane) at a time; the zero
//                      bits of all chunks are kept so that each chunk sees the nearest zero of the chunks
//                      before and after it.  Writes the height and the signed 16-bit offset per voxel.
//   long_axis_kernel   every further axis: lanes run along the contiguous index, a warp takes four
//                      consecutive rows of its 32 columns and scans outward through the read-only cache
//                      until the squared step alone reaches the largest of the four minima.  The site row
//                      is looked for afterwards (the row whose candidate equals the minimum), and only when
//                      a later pass or the index output needs it.
// The scan's cost grows with the distance to the nearest background along the axis; the envelope kernels
// of the generic path do not have that property and stay the choice for everything this path does not take.
#pragma once
#include "edt_wide.cuh"

namespace tmedt {

constexpr uint32_t kLongNoneInt = 0x80000000u;  // above every real height; adding any (n-1)^2 does not wrap
constexpr uint32_t kLongNoneFlt = 0x7f800000u;  // +inf
constexpr int kLongFar = 1 << 20;

template <bool FLT>
__device__ __forceinline__ uint32_t long_add(int d, float w2) {  // the step's own squared length
    if (FLT) return __float_as_uint(__fmul_rn(__fmul_rn(w2, (float)d), (float)d));
    return (uint32_t)(d * d);
}
template <bool FLT>
__device__ __forceinline__ uint32_t long_min(uint32_t v, uint32_t add, uint32_t best) {  // min(best, v + add)
    if (FLT) return min(best, __float_as_uint(__fadd_rn(__uint_as_float(v), __uint_as_float(add))));
    return __viaddmin_u32(v, add, best);
}
template <bool FLT>
__device__ __forceinline__ uint32_t long_cand(uint32_t v, uint32_t add) {
    if (FLT) return __float_as_uint(__fadd_rn(__uint_as_float(v), __uint_as_float(add)));
    return v + add;
}

// First-axis pass.  P.n0 is a multiple of 16 and at most 8192.
template <bool FLT>
__global__ void __launch_bounds__(256) long_row_kernel(const __grid_constant__ WideParams P) {
    constexpr int VPL = 32, CHUNK = 32 * VPL, MAXCH = 8;
    __shared__ uint32_t s_zb[8][MAXCH][32];
    __shared__ int s_first[8][MAXCH], s_last[8][MAXCH];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + warp;
    if (row >= P.rows) return;  // the whole warp leaves together
    const int n0 = P.n0;
    const int nch = (n0 + CHUNK - 1) / CHUNK;
    const uint8_t* src = P.in + row * n0;
    bool row_has_zero = false;
#pragma unroll 1
    for (int c = 0; c < nch; ++c) {
        uint32_t zb = 0u;  // bit b set: voxel b of this lane's 32 is zero
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int x = c * CHUNK + VPL * lane + 16 * h;
            uint4 v = make_uint4(0x01010101u, 0x01010101u, 0x01010101u, 0x01010101u);
            if (x < n0) v = *reinterpret_cast<const uint4*>(src + x);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t m = ~(((w[i] & 0x7f7f7f7fu) + 0x7f7f7f7fu) | w[i]) & 0x80808080u;
                zb |= ((((m >> 7) * 0x00204081u) >> 21) & 0xfu) << (16 * h + 4 * i);
            }
        }
        s_zb[warp][c][lane] = zb;
        const unsigned any = __ballot_sync(0xffffffffu, zb != 0u);
        const int Lf = any ? __ffs(any) - 1 : 0, Ll = any ? 31 - __clz(any) : 0;
        const int fz = __shfl_sync(0xffffffffu, zb ? __ffs(zb) - 1 : 0, Lf);
        const int lz = __shfl_sync(0xffffffffu, zb ? 31 - __clz(zb) : 0, Ll);
        if (lane == 0) {
            s_first[warp][c] = any ? c * CHUNK + VPL * Lf + fz : kLongFar;
            s_last[warp][c] = any ? c * CHUNK + VPL * Ll + lz : -kLongFar;
        }
        row_has_zero |= any != 0u;
    }
    __syncwarp();
    int carry_l = -kLongFar;  // last zero of the chunks before c
#pragma unroll 1
    for (int c = 0; c < nch; ++c) {
        int carry_r = kLongFar;  // first zero of the chunks after c
        for (int c2 = nch - 1; c2 > c; --c2) carry_r = min(carry_r, s_first[warp][c2]);
        const uint32_t zb = s_zb[warp][c][lane];
        const unsigned any = __ballot_sync(0xffffffffu, zb != 0u);
        const int lzin = zb ? 31 - __clz(zb) : 0;
        const int fzin = zb ? __ffs(zb) - 1 : 0;
        const unsigned ml = any & ((1u << lane) - 1u);
        const unsigned mr = lane < 31 ? any >> (lane + 1) : 0u;
        const int Ll = ml ? 31 - __clz(ml) : 0;
        const int Lr = mr ? lane + __ffs(mr) : 0;
        const int lz_l = __shfl_sync(0xffffffffu, lzin, Ll);
        const int fz_r = __shfl_sync(0xffffffffu, fzin, Lr);
        const int x0 = c * CHUNK + VPL * lane;
        uint32_t hts[VPL];
        int16_t offs[VPL];
        int dl[VPL];
        int cur = ml ? c * CHUNK + VPL * Ll + lz_l : carry_l;
#pragma unroll
        for (int b = 0; b < VPL; ++b) {
            if ((zb >> b) & 1u) cur = x0 + b;
            dl[b] = x0 + b - cur;
        }
        cur = mr ? c * CHUNK + VPL * Lr + fz_r : carry_r;
#pragma unroll
        for (int b = VPL - 1; b >= 0; --b) {
            if ((zb >> b) & 1u) cur = x0 + b;
            const int dr = cur - (x0 + b);
            const int a = min(dl[b], dr);
            offs[b] = row_has_zero ? (int16_t)(dl[b] <= dr ? -a : a) : (int16_t)-32768;
            hts[b] = !row_has_zero ? (FLT ? kLongNoneFlt : kLongNoneInt)
                                   : (FLT ? __float_as_uint(__fmul_rn(P.w2x, (float)(a * a))) : (uint32_t)(a * a) * P.w0i);
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int x = x0 + 16 * h;
            if (x < n0) {
                uint4* kdst = reinterpret_cast<uint4*>(P.keys + row * n0 + x);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    kdst[i] = make_uint4(hts[16 * h + 4 * i], hts[16 * h + 4 * i + 1], hts[16 * h + 4 * i + 2],
                                         hts[16 * h + 4 * i + 3]);
                if (P.offs) {
                    uint32_t pk[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        pk[i] = (uint32_t)(uint16_t)offs[16 * h + 2 * i] | ((uint32_t)(uint16_t)offs[16 * h + 2 * i + 1] << 16);
                    uint4* odst = reinterpret_cast<uint4*>(P.offs + row * n0 + x);
                    odst[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    odst[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                }
            }
        }
        carry_l = max(carry_l, s_last[warp][c]);
    }
}

// First-axis pass for rows of any length up to 8192 and any alignment: lanes take consecutive voxels, so every
// load and store of the warp is contiguous.  The zero bits of the row are collected as ballot words in shared
// memory (at most 256 of them); a voxel finds its nearest zero to the left and to the right inside its own word
// with __clz / __ffs, and otherwise takes the last zero before / first zero after the word.
// SH > 0: wide-path keys (off^2 << SH | row index along the second axis); SH == 0: plain off^2 with the wide path's
// "no site" value; SH == -1: float32 heights; SH == -2: plain
// integer heights.
template <int SH>
__global__ void __launch_bounds__(256) long_row_any_kernel(const __grid_constant__ WideParams P) {
    constexpr int MAXW = 256;
    __shared__ uint32_t s_word[8][MAXW];
    __shared__ int s_next[8][MAXW];  // first zero after word b
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + warp;
    if (row >= P.rows) return;  // the whole warp leaves together
    constexpr bool FLT = SH == -1;
    const int n0 = P.n0;
    const uint32_t yrow = SH > 0 ? (uint32_t)(row % P.n1) : 0u;
    const int W = (n0 + 31) >> 5;
    const uint8_t* src = P.in + row * n0;
    for (int b = 0; b < W; ++b) {
        const int x = 32 * b + lane;
        const unsigned word = __ballot_sync(0xffffffffu, x < n0 && src[x] == 0);
        if (lane == 0) s_word[warp][b] = word;
    }
    __syncwarp();
    if (lane == 0) {
        int nxt = kLongFar;
        for (int b = W - 1; b >= 0; --b) {
            s_next[warp][b] = nxt;
            const uint32_t word = s_word[warp][b];
            if (word) nxt = 32 * b + __ffs(word) - 1;
        }
    }
    __syncwarp();
    int carry_l = -kLongFar;  // last zero before word b
    bool row_has_zero = false;
    for (int b = 0; b < W; ++b) row_has_zero |= s_word[warp][b] != 0u;
    for (int b = 0; b < W; ++b) {
        const uint32_t word = s_word[warp][b];
        const int x = 32 * b + lane;
        const uint32_t ml = word & (0xffffffffu >> (31 - lane));  // zeros at or before this voxel
        const uint32_t mr = word >> lane;                          // zeros at or after it
        const int zl = ml ? 32 * b + 31 - __clz(ml) : carry_l;
        const int zr = mr ? x + __ffs(mr) - 1 : s_next[warp][b];
        const int dl = x - zl, dr = zr - x;
        const int a = min(dl, dr);
        if (x < n0) {
            if (P.offs) P.offs[row * n0 + x] = row_has_zero ? (int16_t)(dl <= dr ? -a : a) : (int16_t)-32768;
            P.keys[row * n0 + x] = !row_has_zero ? (FLT ? kLongNoneFlt : kLongNoneInt)
                                                 : (FLT ? __float_as_uint(__fmul_rn(P.w2x, (float)(a * a)))
                                                        : ((((uint32_t)(a * a) * (SH == -2 || SH == 0 ? P.w0i : 1u)) << (SH > 0 ? SH : 0)) | yrow));
        }
        if (word) carry_l = 32 * b + 31 - __clz(word);
    }
}

struct LongAxisParams {
    const uint32_t* h_in;      // (outer, n, inner) heights
    const int16_t* offs_in;    // (outer, n, inner, K)
    uint32_t* h_out;           // (outer, n, inner), unused when FINAL
    int16_t* offs_out;         // (outer, n, inner, K + 1), unused when FINAL
    int64_t outer, inner;
    int n;
    int n0;                    // extent of the contiguous axis (to split an inner position into coordinates)
    float w2;                  // squared sampling of this axis (float heights)
    int strips_per_slab;       // ceil(inner / 32)
    int row_blocks;            // ceil(n / kLongRows)
    uint32_t* blockmin;        // (outer, ceil(n / 32), inner): minimum height of every 32 rows, or nullptr (short axes)
};

// Minimum height of every block of 32 consecutive rows of every column.
__global__ void __launch_bounds__(256) long_blockmin_kernel(const __grid_constant__ LongAxisParams P) {
    const int nblk = (P.n + 31) >> 5;
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= P.outer * nblk * P.inner) return;
    const int64_t c = t % P.inner, sb = t / P.inner;
    const int B = (int)(sb % nblk);
    const int64_t slab = sb / nblk;
    const uint32_t* col = P.h_in + slab * (int64_t)P.n * P.inner + c;
    uint32_t m = 0xffffffffu;
    const int r1 = min(P.n, 32 * B + 32);
    for (int r = 32 * B; r < r1; ++r) m = min(m, __ldg(col + (int64_t)r * P.inner));
    P.blockmin[t] = m;
}

constexpr int kLongRows = 256;  // rows of a strip one block handles

template <int K, bool FINAL, bool FLT>
__global__ void __launch_bounds__(256) long_axis_kernel(const __grid_constant__ LongAxisParams P,
                                                        const __grid_constant__ EpilogueParams ep) {
    constexpr uint32_t NONE = FLT ? kLongNoneFlt : kLongNoneInt;
    constexpr int R = 4;
    const int n = P.n;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const unsigned rb = blockIdx.x % (unsigned)P.row_blocks;
    const unsigned sb = blockIdx.x / (unsigned)P.row_blocks;
    const unsigned strip = sb % (unsigned)P.strips_per_slab;
    const int64_t slab = sb / (unsigned)P.strips_per_slab;
    const int64_t c = (int64_t)strip * 32 + lane;  // position along inner
    if (c >= P.inner) return;
    const int64_t slab_base = slab * (int64_t)n * P.inner;
    const int64_t col_base = slab_base + c;
    const uint32_t* __restrict__ col = P.h_in + col_base;
    const int64_t st = P.inner;
    const int cx = (int)(c % P.n0), cy = (int)(c / P.n0);
    const int y_end = min(n, (int)(rb + 1) * kLongRows);
    // the warps of a block work on neighbouring groups of rows at any time, so that their reads overlap in cache
    for (int y0 = (int)rb * kLongRows + warp * R; y0 < y_end; y0 += nwarps * R) {
        uint32_t v[R], best[R];
#pragma unroll
        for (int i = 0; i < R; ++i) v[i] = y0 + i < n ? __ldg(col + (int64_t)(y0 + i) * st) : NONE;
#pragma unroll
        for (int i = 0; i < R; ++i) {
            best[i] = v[i];
#pragma unroll
            for (int j = 0; j < R; ++j)
                if (j != i) best[i] = long_min<FLT>(v[j], long_add<FLT>(i - j, P.w2), best[i]);
            if (y0 + i >= n) best[i] = 0u;
        }
        uint32_t mx = max(max(best[0], best[1]), max(best[2], best[3]));
        // Near phase: outward, row by row, over the group's own block of 32 rows and the two next to it (the
        // whole column when there are no block minima).  Far phase: block by block, nearest first; a block is
        // read only if its minimum height plus the squared distance to its nearest row could still lower one
        // of the four minima.  blk[i]: far block in which minimum i was last lowered (-1: near phase).
        const int Bg = y0 >> 5, nblk = (n + 31) >> 5;
        const int lo_min = P.blockmin ? max(0, (Bg - 1) * 32) : 0;
        const int hi_max = P.blockmin ? min(n - 1, (Bg + 2) * 32 - 1) : n - 1;
        int blk[R] = {-1, -1, -1, -1};
        if (mx != 0u) {
            int lo = y0 - 1, hi = y0 + R;
            const uint32_t* plo = col + (int64_t)lo * st;
            const uint32_t* phi = col + (int64_t)hi * st;
            for (int d = 1; lo >= lo_min || hi <= hi_max; ++d, --lo, ++hi, plo -= st, phi += st) {
                if (long_add<FLT>(d, P.w2) >= mx) break;
                const uint32_t vlo = lo >= lo_min ? __ldg(plo) : NONE;
                const uint32_t vhi = hi <= hi_max ? __ldg(phi) : NONE;
#pragma unroll
                for (int i = 0; i < R; ++i) {
                    best[i] = long_min<FLT>(vlo, long_add<FLT>(d + i, P.w2), best[i]);
                    best[i] = long_min<FLT>(vhi, long_add<FLT>(d + R - 1 - i, P.w2), best[i]);
                }
                mx = max(max(best[0], best[1]), max(best[2], best[3]));
            }
            // (the near phase may stop on one side's range before the other's: the far phase tests each side itself)
            if (P.blockmin) {
                const uint32_t* bm = P.blockmin + slab * (int64_t)nblk * st + c;
                for (int k = 2; Bg - k >= 0 || Bg + k < nblk; ++k) {
                    const int dlo = y0 - (32 * (Bg - k) + 31), dhi = 32 * (Bg + k) - (y0 + R - 1);
                    const bool in_lo = Bg - k >= 0 && long_add<FLT>(dlo, P.w2) < mx;
                    const bool in_hi = Bg + k < nblk && long_add<FLT>(dhi, P.w2) < mx;
                    if (!in_lo && !in_hi) break;  // both distances only grow from here
#pragma unroll
                    for (int side = 0; side < 2; ++side) {
                        if (!(side ? in_hi : in_lo)) continue;
                        const int B = side ? Bg + k : Bg - k;
                        const uint32_t m = __ldg(bm + (int64_t)B * st);
                        if (long_cand<FLT>(m, long_add<FLT>(side ? dhi : dlo, P.w2)) >= mx) continue;
                        const int r1 = min(n, 32 * B + 32);
                        uint32_t old[R];
#pragma unroll
                        for (int i = 0; i < R; ++i) old[i] = best[i];
                        for (int r = 32 * B; r < r1; ++r) {
                            const uint32_t vr = __ldg(col + (int64_t)r * st);
#pragma unroll
                            for (int i = 0; i < R; ++i)
                                best[i] = long_min<FLT>(vr, long_add<FLT>(y0 + i - r, P.w2), best[i]);
                        }
#pragma unroll
                        for (int i = 0; i < R; ++i)
                            if (best[i] != old[i]) blk[i] = B;
                        mx = max(max(best[0], best[1]), max(best[2], best[3]));
                    }
                }
            }
        }
        const bool need_site = FINAL ? ep.idx != nullptr : P.offs_out != nullptr;
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int y = y0 + i;
            if (y >= n) break;
            const uint32_t b = best[i];
            const bool none = b >= NONE;
            int j = y;
            if (need_site && !none) {
                // the minimum is attained: find a row whose candidate equals it
                if (blk[i] < 0) {
                    for (int d = 0; d < n; ++d) {
                        const uint32_t add = long_add<FLT>(d, P.w2);
                        if (y - d >= 0 && long_cand<FLT>(__ldg(col + (int64_t)(y - d) * st), add) == b) { j = y - d; break; }
                        if (y + d < n && long_cand<FLT>(__ldg(col + (int64_t)(y + d) * st), add) == b) { j = y + d; break; }
                    }
                } else {
                    const int r1 = min(n, 32 * blk[i] + 32);
                    for (int r = 32 * blk[i]; r < r1; ++r)
                        if (long_cand<FLT>(__ldg(col + (int64_t)r * st), long_add<FLT>(y - r, P.w2)) == b) { j = r; break; }
                }
            }
            const int64_t p = col_base + (int64_t)y * st;    // this voxel
            const int64_t pj = col_base + (int64_t)j * st;   // the chosen site's voxel of this column
            if (!FINAL) {
                P.h_out[p] = none ? NONE : b;
                if (K == 1 && P.offs_out) {
                    const uint32_t o0 = none ? 0x8000u : (uint32_t)(uint16_t)P.offs_in[pj];
                    reinterpret_cast<uint32_t*>(P.offs_out)[p] = o0 | ((uint32_t)(uint16_t)(int16_t)(j - y) << 16);
                }
            } else {
                if (ep.dist)
                    ep.dist[p] = none ? TMEDT_INF : __fsqrt_rn(FLT ? __uint_as_float(b) : (float)b);
                if (ep.sq) ep.sq[p] = none ? INT64_MAX : (int64_t)b;  // unit sampling only
                if (ep.idx) {
                    int site[3] = {0, 0, 0};
                    if (!none) {
                        if (K == 1) {
                            site[0] = cx + (int)P.offs_in[pj];
                            site[1] = j;
                        } else {
                            const uint32_t o = reinterpret_cast<const uint32_t*>(P.offs_in)[pj];
                            site[0] = cx + (int)(int16_t)(o & 0xffffu);
                            site[1] = cy + (int)(int16_t)(o >> 16);
                            site[2] = j;
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
                        int64_t val = 0;
#pragma unroll
                        for (int q = 0; q <= K; ++q)
                            if (a == ep.axis[q]) val = site[q];
                        ep.idx[(slab * ep.ndim + a) * ep.V + vox] = none ? -1 : val;
                    }
                }
            }
        }
    }
}

}  // namespace tmedt
