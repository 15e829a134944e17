// Rank- and extent-generic kernels: the first-axis pass on bit-packed lines and one lower-envelope
// pass per further axis.  They cover every supported shape; faster specialised kernels replace
// them where the planner can use those.
#pragma once
#include "edt_common.cuh"

namespace tmedt {

// ---------------------------------------------------------------------------------------------
// First-axis pass (contiguous axis).  For every voxel of a line of length n: the signed offset to the
// nearest zero voxel of the same line (left wins ties), or the "none" sentinel when the line has no
// zero.  The zero flags of 32 consecutive voxels are packed into a word with a warp ballot; inside the
// word the nearest zero to the left is 31 - clz(word & mask_up_to_lane) and to the right
// lane + ffs(word >> lane) - 1; across words the last zero before / first zero after each word come
// from a running scan over the words of the line.
// ---------------------------------------------------------------------------------------------
struct Pass0Params {
    const uint8_t* in;  // (lines, n)
    void* out;          // plane 0, (lines, n) of OT; unused when FINAL
    int64_t lines;
    int n;
    double w;           // sampling of this axis (FINAL only)
};

template <typename OT>
__device__ __forceinline__ void pass0_store(const Pass0Params& P, const EpilogueParams& ep, bool final_pass,
                                            int64_t line, int x, int lp, int rp) {
    // lp: position of nearest zero at or left of x, or -1; rp: at or right of x, or INT_MAX.
    int off;
    bool none = false;
    if (lp < 0 && rp == INT_MAX) { none = true; off = OffTraits<OT>::kNone; }
    else if (lp < 0) off = rp - x;
    else if (rp == INT_MAX) off = lp - x;
    else off = (x - lp <= rp - x) ? (lp - x) : (rp - x);
    if (!final_pass) {
        reinterpret_cast<OT*>(P.out)[line * (int64_t)P.n + x] = (OT)off;
    } else {
        // Single processed axis: every other axis has extent 1, so the line is the image.
        const int64_t e = line * ep.V + x;
        if (none) {
            if (ep.dist) ep.dist[e] = __int_as_float(0x7f800000);
            if (ep.sq) ep.sq[e] = INT64_MAX;
            if (ep.idx && ep.flat) ep.idx[e] = -1;
            else if (ep.idx)
                for (int a = 0; a < ep.ndim; ++a) ep.idx[(line * ep.ndim + a) * ep.V + x] = -1;
        } else {
            const int ao = off < 0 ? -off : off;
            if (ep.dist) ep.dist[e] = (float)(P.w * (double)ao);
            if (ep.sq) ep.sq[e] = (int64_t)ao * ao;
            if (ep.idx && ep.flat) ep.idx[e] = (int64_t)(x + off) * ep.pstride[0];
            else if (ep.idx)
                for (int a = 0; a < ep.ndim; ++a)
                    ep.idx[(line * ep.ndim + a) * ep.V + x] = (a == ep.axis[0]) ? (int64_t)(x + off) : 0;
        }
    }
}

// n <= 32: floor(32 / n) whole lines share one ballot word.
template <typename OT, bool FINAL>
__global__ void __launch_bounds__(256) pass0_short_kernel(const __grid_constant__ Pass0Params P,
                                                          const __grid_constant__ EpilogueParams ep) {
    const int n = P.n;
    const int per_warp = 32 / n;
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int sub = lane / n, pos = lane - sub * n;
    const int64_t line = warp * per_warp + sub;
    const bool valid = sub < per_warp && line < P.lines;
    uint8_t b = 1;
    if (valid) b = P.in[line * n + pos];
    const unsigned Z = __ballot_sync(0xffffffffu, valid && b == 0);
    if (!valid) return;
    const unsigned seg = ((n == 32) ? 0xffffffffu : ((1u << n) - 1u)) << (sub * n);
    const unsigned Zs = Z & seg;
    const unsigned Zl = Zs & (0xffffffffu >> (31 - lane));
    const unsigned Zr = Zs >> lane;
    const int base = sub * n;
    const int lp = Zl ? (31 - __clz(Zl)) - base : -1;
    const int rp = Zr ? (lane + __ffs(Zr) - 1) - base : INT_MAX;
    pass0_store<OT>(P, ep, FINAL, line, pos, lp, rp);
}

// n > 32: one warp per line.  Shared memory per warp: nw words of zero flags, nw "last zero before this
// word" and nw "first zero after this word" entries (nw = ceil(n / 32)).
template <typename OT, bool FINAL>
__global__ void __launch_bounds__(128) pass0_long_kernel(const __grid_constant__ Pass0Params P,
                                                         const __grid_constant__ EpilogueParams ep) {
    extern __shared__ int sm_pass0[];
    const int n = P.n;
    const int nw = (n + 31) >> 5;
    const int lane = threadIdx.x & 31;
    const int wib = threadIdx.x >> 5;
    const int64_t line = (int64_t)blockIdx.x * (blockDim.x >> 5) + wib;
    if (line >= P.lines) return;  // whole warp leaves together
    unsigned* Zw = reinterpret_cast<unsigned*>(sm_pass0) + (size_t)wib * 3 * nw;
    int* prevw = reinterpret_cast<int*>(Zw) + nw;
    int* nextw = prevw + nw;
    const uint8_t* row = P.in + line * (int64_t)n;
    for (int w = 0; w < nw; ++w) {
        const int x = w * 32 + lane;
        const uint8_t b = x < n ? row[x] : (uint8_t)1;
        const unsigned Z = __ballot_sync(0xffffffffu, x < n && b == 0);
        if (lane == 0) Zw[w] = Z;
    }
    __syncwarp();
    // last zero strictly before each word (forward) and first zero strictly after it (backward)
    int carry = -1;
    for (int w0 = 0; w0 < nw; w0 += 32) {
        const int w = w0 + lane;
        const unsigned Z = w < nw ? Zw[w] : 0u;
        int last = Z ? w * 32 + 31 - __clz(Z) : -1;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, last, d);
            if (lane >= d) last = max(last, o);
        }
        int excl = __shfl_up_sync(0xffffffffu, last, 1);
        if (lane == 0) excl = -1;
        if (w < nw) prevw[w] = max(excl, carry);
        carry = max(carry, __shfl_sync(0xffffffffu, last, 31));
    }
    carry = INT_MAX;
    for (int w0 = ((nw - 1) / 32) * 32; w0 >= 0; w0 -= 32) {
        const int w = w0 + lane;
        const unsigned Z = w < nw ? Zw[w] : 0u;
        int first = Z ? w * 32 + __ffs(Z) - 1 : INT_MAX;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_down_sync(0xffffffffu, first, d);
            if (lane + d < 32) first = min(first, o);
        }
        int excl = __shfl_down_sync(0xffffffffu, first, 1);
        if (lane == 31) excl = INT_MAX;
        if (w < nw) nextw[w] = min(excl, carry);
        carry = min(carry, __shfl_sync(0xffffffffu, first, 0));
    }
    __syncwarp();
    for (int w = 0; w < nw; ++w) {
        const int x = w * 32 + lane;
        if (x >= n) break;
        const unsigned Z = Zw[w];
        const unsigned Zl = Z & (0xffffffffu >> (31 - lane));
        const unsigned Zr = Z >> lane;
        const int lp = Zl ? w * 32 + 31 - __clz(Zl) : prevw[w];
        const int rp = Zr ? x + __ffs(Zr) - 1 : nextw[w];
        pass0_store<OT>(P, ep, FINAL, line, x, lp, rp);
    }
}

// ---------------------------------------------------------------------------------------------
// Lower-envelope pass along a strided axis, one thread per line, lanes along the contiguous
// `inner` index so every load and store of a warp is a contiguous run.
//
// The array is viewed as (outer, n, inner).  Sites are the voxels of the line that already have a
// nearest background voxel with respect to the earlier axes; site s has height h_s = sum over earlier
// planes of w_q^2 off_q^2 and contributes the parabola F_s(x) = h_s + w^2 (x - s)^2.  The pass takes,
// at every integer x of the line, the site with the least F_s(x).
//
// The envelope is kept as a stack of (site s_k, start t_k): site s_k is the minimiser on the integer
// interval [t_k, t_{k+1}).  Both sequences increase strictly with k, so the stack is stored as two
// bit masks over the line positions (bit s set = s is on the stack; bit t set = an interval starts at
// t); the k-th set bit of one pairs with the k-th set bit of the other.  Push sets the next higher bit
// in each, pop clears the highest, and the query walks both masks upward.  The top entry is cached
// in registers.  A new site u pops the top while F_top(t_top) > F_u(t_top) (u is then better on all of
// the top's interval), and otherwise starts its own interval right after the last x where the top is
// still at least as good:  x* = (h_u - h_top) / (2 w^2 (u - s_top)) + (u + s_top) / 2,
// t_u = floor(x*) + 1, dropped when t_u >= n.
// ---------------------------------------------------------------------------------------------
struct AxisParams {
    const void* in;   // K planes of OT, plane stride = plane_elems
    void* out;        // K + 1 planes of OT (unused when FINAL)
    int64_t plane_elems;
    int64_t lines;    // outer * inner
    int64_t inner;
    int n;
    double w2;        // squared sampling of this axis
    double w2p[kMaxDims];  // squared sampling of the earlier planes
};

template <typename CT, typename OT, int K>
__device__ __forceinline__ bool load_site(const OT* __restrict__ in, int64_t plane_elems, int64_t e,
                                          const CT* w2p, CT& h, int* off) {
    const int o0 = in[e];
    if (o0 == OffTraits<OT>::kNone) return false;
    off[0] = o0;
    h = w2p[0] * (CT)o0 * (CT)o0;
#pragma unroll
    for (int p = 1; p < K; ++p) {
        const int o = in[p * plane_elems + e];
        off[p] = o;
        h += w2p[p] * (CT)o * (CT)o;
    }
    return true;
}

__device__ __forceinline__ int mask_highest_below(const unsigned* m, int stride, int pos) {
    // highest set bit strictly below `pos`, or -1
    int w = pos >> 5;
    unsigned word = m[w * stride] & ((1u << (pos & 31)) - 1u);
    while (word == 0u) {
        if (--w < 0) return -1;
        word = m[w * stride];
    }
    return w * 32 + 31 - __clz(word);
}

__device__ __forceinline__ int mask_lowest_above(const unsigned* m, int stride, int nw, int pos) {
    // lowest set bit strictly above `pos` (pos may be -1), or -1
    int p = pos + 1;
    int w = p >> 5;
    if (w >= nw) return -1;
    unsigned word = m[w * stride] & (0xffffffffu << (p & 31));
    while (word == 0u) {
        if (++w >= nw) return -1;
        word = m[w * stride];
    }
    return w * 32 + __ffs(word) - 1;
}

template <typename CT, typename OT, int K, bool FINAL>
__global__ void __launch_bounds__(128) axis_pass_kernel(const __grid_constant__ AxisParams P,
                                                        const __grid_constant__ EpilogueParams ep) {
    extern __shared__ unsigned sm_axis[];
    const int T = blockDim.x;
    const int n = P.n;
    const int nw = (n + 31) >> 5;
    unsigned* S = sm_axis + threadIdx.x;
    unsigned* Tm = sm_axis + (size_t)nw * T + threadIdx.x;
    const int64_t line = (int64_t)blockIdx.x * T + threadIdx.x;
    if (line >= P.lines) return;
    const int64_t o = line / P.inner, r = line - o * P.inner;
    const int64_t base = o * (int64_t)n * P.inner + r;
    const OT* __restrict__ in = reinterpret_cast<const OT*>(P.in);
    const CT w2 = (CT)P.w2;
    const CT inv2w2 = (CT)(0.5 / P.w2);
    CT w2p[K];
#pragma unroll
    for (int p = 0; p < K; ++p) w2p[p] = (CT)P.w2p[p];

    for (int w = 0; w < nw; ++w) { S[w * T] = 0u; Tm[w * T] = 0u; }

    // ---- build the envelope ----
    int s_top = -1, t_top = 0;
    CT h_top = 0;
    int offs[K];
    for (int u = 0; u < n; ++u) {
        CT hu;
        if (!load_site<CT, OT, K>(in, P.plane_elems, base + (int64_t)u * P.inner, w2p, hu, offs)) continue;
        int t_new = 0;
        bool push = true;
        while (s_top >= 0) {
            const CT a = (CT)(t_top - s_top), b = (CT)(t_top - u);
            const CT ft = h_top + w2 * a * a, fu = hu + w2 * b * b;
            if (ft > fu) {  // u beats the top on the whole of the top's interval: pop
                S[(s_top >> 5) * T] &= ~(1u << (s_top & 31));
                Tm[(t_top >> 5) * T] &= ~(1u << (t_top & 31));
                const int s_prev = mask_highest_below(S, T, s_top);
                if (s_prev < 0) { s_top = -1; break; }
                t_top = mask_highest_below(Tm, T, t_top);
                s_top = s_prev;
                int dummy[K];
                load_site<CT, OT, K>(in, P.plane_elems, base + (int64_t)s_top * P.inner, w2p, h_top, dummy);
                continue;
            }
            const CT xs = (hu - h_top) * inv2w2 / (CT)(u - s_top) + (CT)(u + s_top) * (CT)0.5;
            if (xs < (CT)(n - 1)) {
                t_new = (int)floor(xs) + 1;
                if (t_new <= t_top) t_new = t_top + 1;  // rounding guard: starts stay strictly increasing
                push = t_new < n;
            } else {
                push = false;
            }
            break;
        }
        if (push) {
            S[(u >> 5) * T] |= 1u << (u & 31);
            Tm[(t_new >> 5) * T] |= 1u << (t_new & 31);
            s_top = u; t_top = t_new; h_top = hu;
        }
    }

    // ---- query ----
    OT* out = reinterpret_cast<OT*>(P.out);
    int coord[kMaxDims];
    int64_t vimg = 0;
    if (FINAL) {
        // The last pass runs along the first processed spatial axis, so `o` is the image index and
        // r enumerates the later axes, plane 0 fastest.
        int64_t rr = r;
#pragma unroll
        for (int p = 0; p < K; ++p) { coord[p] = (int)(rr % ep.ext[p]); rr /= ep.ext[p]; }
        vimg = r;
    }
    int s_cur = mask_lowest_above(S, T, nw, -1);
    if (s_cur < 0) {  // no site on this line
        for (int i = 0; i < n; ++i) {
            const int64_t e = base + (int64_t)i * P.inner;
            if (!FINAL) {
                out[e] = (OT)OffTraits<OT>::kNone;
#pragma unroll
                for (int p = 1; p <= K; ++p) out[p * P.plane_elems + e] = 0;
            } else {
                emit_outputs<CT>(ep, o, vimg + (int64_t)i * P.inner, coord, offs, true);
            }
        }
        return;
    }
    CT hdummy;
    load_site<CT, OT, K>(in, P.plane_elems, base + (int64_t)s_cur * P.inner, w2p, hdummy, offs);
    unsigned wT = 0;
    for (int i = 0; i < n; ++i) {
        if ((i & 31) == 0) wT = Tm[(i >> 5) * T];
        if (i > 0 && ((wT >> (i & 31)) & 1u)) {
            s_cur = mask_lowest_above(S, T, nw, s_cur);
            load_site<CT, OT, K>(in, P.plane_elems, base + (int64_t)s_cur * P.inner, w2p, hdummy, offs);
        }
        const int64_t e = base + (int64_t)i * P.inner;
        if (!FINAL) {
#pragma unroll
            for (int p = 0; p < K; ++p) out[p * P.plane_elems + e] = (OT)offs[p];
            out[K * P.plane_elems + e] = (OT)(s_cur - i);
        } else {
            int fo[kMaxDims];
#pragma unroll
            for (int p = 0; p < K; ++p) fo[p] = offs[p];
            fo[K] = s_cur - i;
            coord[K] = i;
            emit_outputs<CT>(ep, o, vimg + (int64_t)i * P.inner, coord, fo, false);
        }
    }
}

}  // namespace tmedt
