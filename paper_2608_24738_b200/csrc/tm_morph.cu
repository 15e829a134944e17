// tm_morph: host side of the fused erosion / dilation kernel (see include/tm_morph.h and morph.cuh).
// Flattens the structuring element into its active entries, reflects it for a dilation (with the origin rule of
// scipy.ndimage for even sizes), computes the per-axis offset extrema for the interior test, copies the entry
// list to the device and launches one kernel.
#include <math.h>
#include <string.h>

#include <algorithm>
#include <vector>

#include "../../include/tm_morph.h"
#include "host_shared.h"
#include "morph.cuh"
#include "morph_bits.cuh"
#include "morph_box.cuh"

using namespace tmmorph;

namespace {

struct Geometry {
    int ndim;
    int64_t images, V, total;
    int ext[kMaxDims], stride[kMaxDims];
};

int check_geometry(int ndim, const int64_t* shape, Geometry& g) {
    if (ndim < 1 || ndim > kMaxDims || !shape) return TM_EDT_ERR_INVALID_ARG;
    g.ndim = ndim;
    if (shape[0] < 0 || shape[1] < 0) return TM_EDT_ERR_INVALID_ARG;
    g.images = shape[0] * shape[1];
    g.V = 1;
    for (int a = 0; a < ndim; ++a) {
        if (shape[2 + a] < 0) return TM_EDT_ERR_INVALID_ARG;
        if (shape[2 + a] > 0 && g.V > (int64_t)INT32_MAX / shape[2 + a]) return TM_EDT_ERR_UNSUPPORTED;  // int offsets
        g.V *= shape[2 + a];
    }
    if (g.images > 0 && g.V > 0 && g.images > ((int64_t)1 << 40) / g.V) return TM_EDT_ERR_UNSUPPORTED;
    g.total = g.images * g.V;
    int64_t st = 1;
    for (int a = ndim - 1; a >= 0; --a) {
        g.ext[a] = (int)shape[2 + a];
        g.stride[a] = (int)st;
        st *= shape[2 + a];
    }
    return TM_EDT_OK;
}

// Active entries of the element, for an erosion-style combine out(x) = op_k f(x + k - c).  A dilation is the same
// combine with the element reflected through its centre and the origin negated (minus one on even sizes).
int flatten(const Geometry& g, const uint8_t* fp, const float* st, const int64_t* fp_shape, const int64_t* origin,
            bool reflect, std::vector<Entry>& out, int* lo, int* hi) {
    if (!fp || !fp_shape) return TM_EDT_ERR_INVALID_ARG;
    int m[kMaxDims], c[kMaxDims];
    int64_t count = 1;
    for (int a = 0; a < g.ndim; ++a) {
        if (fp_shape[a] < 1 || fp_shape[a] > 255) return TM_EDT_ERR_INVALID_ARG;
        m[a] = (int)fp_shape[a];
        int64_t o = origin ? origin[a] : 0;
        if (reflect) o = -o - (m[a] % 2 == 0 ? 1 : 0);
        const int64_t centre = m[a] / 2 + o;
        if (centre < 0 || centre >= m[a]) return TM_EDT_ERR_INVALID_ARG;
        c[a] = (int)centre;
        count *= m[a];
        if (count > (int64_t)1 << 24) return TM_EDT_ERR_UNSUPPORTED;
        lo[a] = INT32_MAX; hi[a] = INT32_MIN;
    }
    int k[kMaxDims] = {0};
    for (int64_t i = 0; i < count; ++i) {
        // position k of the (possibly reflected) element <- position m - 1 - k of the caller's array
        int64_t src = 0;
        for (int a = 0; a < g.ndim; ++a) src = src * m[a] + (reflect ? m[a] - 1 - k[a] : k[a]);
        if (fp[src] != 0) {
            if ((int)out.size() >= TM_MORPH_MAX_ENTRIES) return TM_EDT_ERR_UNSUPPORTED;
            Entry en;
            memset(&en, 0, sizeof(en));
            for (int a = 0; a < g.ndim; ++a) {
                const int off = k[a] - c[a];
                en.off[a] = (int16_t)off;
                en.flat += off * g.stride[a];
                lo[a] = off < lo[a] ? off : lo[a];
                hi[a] = off > hi[a] ? off : hi[a];
            }
            en.s = st ? st[src] : 0.0f;
            out.push_back(en);
        }
        for (int a = g.ndim - 1; a >= 0; --a) {
            if (++k[a] < m[a]) break;
            k[a] = 0;
        }
    }
    return out.empty() ? TM_EDT_ERR_INVALID_ARG : TM_EDT_OK;
}

template <typename T, bool BINARY>
int run(const T* input, int ndim, const int64_t* shape, const uint8_t* fp, const float* st, const int64_t* fp_shape,
        const int64_t* origin, int op, int mode, float cval, int border_value, void* output, tm_edt_stream_t stream,
        bool allow_separable = true);

// A flat element whose footprint is a full box is the composition of one line element per axis: the minimum (or
// maximum) over a box is the minimum over its rows of the minima along the rows, and every border rule acts on one
// axis at a time.  From 20 positions on, the box is therefore run as one pass per axis with ndim line elements
// (m_0 + .. + m_{d-1} taps instead of their product), through the same kernels, with one or two scratch images.
template <typename T, bool BINARY>
int run_box(const T* input, int ndim, const int64_t* shape, const int64_t* fp_shape, const int64_t* origin, int op,
            int mode, float cval, int border_value, void* output, tm_edt_stream_t stream, size_t total) {
    cudaStream_t s = (cudaStream_t)stream;
    int axes[kMaxDims], na = 0;
    for (int a = 0; a < ndim; ++a)
        if (fp_shape[a] > 1 || (origin && origin[a] != 0)) axes[na++] = a;
    if (na == 0) axes[na++] = ndim - 1;
    const size_t buf = ((total * sizeof(T)) + 255) & ~(size_t)255;
    char* ws = nullptr;
    if (na > 1) {
        cudaError_t e = tmedt::shared_scratch_alloc((void**)&ws, (na > 2 ? 2 : 1) * buf, s);
        if (e != cudaSuccess) { cudaGetLastError(); tmedt::shared_record((int)e, 0); return TM_EDT_ERR_ALLOC; }
    }
    uint8_t line[256];
    memset(line, 1, sizeof(line));
    const T* src = input;
    int rc = TM_EDT_OK, launches = 0;
    for (int i = 0; i < na && rc == TM_EDT_OK; ++i) {
        const int a = axes[i];
        int64_t ls[kMaxDims], lo[kMaxDims];
        for (int b = 0; b < ndim; ++b) { ls[b] = b == a ? fp_shape[b] : 1; lo[b] = (b == a && origin) ? origin[b] : 0; }
        void* dst = i == na - 1 ? output : (void*)(ws + (size_t)(i & 1) * buf);
        rc = run<T, BINARY>(src, ndim, shape, line, nullptr, ls, lo, op, mode, cval, border_value, dst, stream, false);
        launches += 2;
        src = static_cast<const T*>(dst);
    }
    if (ws) cudaFreeAsync(ws, s);
    if (rc == TM_EDT_OK) tmedt::shared_record(-1, launches);
    return rc;
}

// One pass of box_strip_kernel: a window of +-rh along the contiguous axis and +-rv along the walk axis.
static bool launch_box_strip(bool ero, int rh, int rv, const StripParams& B, unsigned blocks, cudaStream_t s) {
#define TM_BOX_STRIP(RH, RV)                                                                                     \
    do {                                                                                                         \
        if (ero) box_strip_kernel<true, RH, RV, box_strip_len(RV)><<<blocks, dim3(32, 8), 0, s>>>(B);             \
        else box_strip_kernel<false, RH, RV, box_strip_len(RV)><<<blocks, dim3(32, 8), 0, s>>>(B);                \
        return true;                                                                                             \
    } while (0)
    if (rh == rv) { switch (rh) { case 1: TM_BOX_STRIP(1, 1); case 2: TM_BOX_STRIP(2, 2); case 3: TM_BOX_STRIP(3, 3); case 4: TM_BOX_STRIP(4, 4); } }
    else if (rv == 0) { switch (rh) { case 1: TM_BOX_STRIP(1, 0); case 2: TM_BOX_STRIP(2, 0); case 3: TM_BOX_STRIP(3, 0); case 4: TM_BOX_STRIP(4, 0); } }
    else if (rh == 0) { switch (rv) { case 1: TM_BOX_STRIP(0, 1); case 2: TM_BOX_STRIP(0, 2); case 3: TM_BOX_STRIP(0, 3); case 4: TM_BOX_STRIP(0, 4); } }
#undef TM_BOX_STRIP
    return false;
}

// A flat full box of odd extents (at most 9 per axis), centred on its voxel, on a float32 image: passes of
// box_strip_kernel (morph_box.cuh), the last two axes in one pass when their extents are equal, one further pass per
// earlier axis; every border rule is applied inside the kernel.  Returns -1 when the shape or the element does not
// fit, and the caller goes on with the general kernels.
static int run_box_quads(const float* input, int ndim, const int64_t* fp_shape, const int64_t* origin,
                         int op, int mode, float cval, float* output, tm_edt_stream_t stream, const Geometry& g) {
    const int nd = ndim, W = g.ext[nd - 1];
    if (W % 4 != 0 || ((uintptr_t)input & 15u) || ((uintptr_t)output & 15u)) return -1;
    int rad[kMaxDims];
    for (int a = 0; a < nd; ++a) {
        const int m = (int)fp_shape[a];
        if (m % 2 == 0 || m > 9 || (origin && origin[a] != 0)) return -1;
        rad[a] = m / 2;
    }
    // passes as (radius along the row, walk axis, radius along it); walk axis -1: no walk
    struct Pass { int rh, axis, rv; } pass[kMaxDims + 1];
    int np = 0;
    const int rh = rad[nd - 1], rv = nd >= 2 ? rad[nd - 2] : 0;
    if (rh == rv || rh == 0 || rv == 0) { if (rh || rv) pass[np++] = {rh, nd >= 2 ? nd - 2 : -1, rv}; }
    else { pass[np++] = {rh, nd >= 2 ? nd - 2 : -1, 0}; pass[np++] = {0, nd - 2, rv}; }
    for (int a = nd - 3; a >= 0; --a)
        if (rad[a]) pass[np++] = {0, a, rad[a]};
    if (np == 0) return -1;
    for (int i = 0; i < np; ++i) {  // every pass must fit a grid before the first one is launched
        const int n = pass[i].axis >= 0 ? g.ext[pass[i].axis] : 1, T = box_strip_len(pass[i].rv);
        const int64_t blocks = g.total / ((int64_t)n * W) * (((n + T - 1) / T + 7) / 8) * ((W / 4 + 31) / 32);
        if (blocks > (int64_t)INT32_MAX) return -1;
    }
    cudaStream_t s = (cudaStream_t)stream;
    const size_t buf = (((size_t)g.total * 4) + 255) & ~(size_t)255;
    char* ws = nullptr;
    if (np > 1) {
        cudaError_t e = tmedt::shared_scratch_alloc((void**)&ws, (np > 2 ? 2 : 1) * buf, s);
        if (e != cudaSuccess) { cudaGetLastError(); tmedt::shared_record((int)e, 0); return TM_EDT_ERR_ALLOC; }
    }
    const float* src = input;
    int rc = TM_EDT_OK, launches = 0;
    for (int i = 0; i < np && rc == TM_EDT_OK; ++i) {
        float* dst = i == np - 1 ? output : reinterpret_cast<float*>(ws + (size_t)(i & 1) * buf);
        StripParams B;
        memset(&B, 0, sizeof(B));
        B.in = src; B.out = dst; B.W = W; B.mode = mode; B.cval = cval; B.reverse = i & 1;
        B.chunks = (unsigned)((W / 4 + 31) / 32);
        if (pass[i].axis >= 0) { B.n = g.ext[pass[i].axis]; B.walk_stride = g.stride[pass[i].axis]; }
        else { B.n = 1; B.walk_stride = W; }
        B.inner = (int)(B.walk_stride / W);
        const int T = box_strip_len(pass[i].rv);
        B.strip_groups = (unsigned)(((B.n + T - 1) / T + 7) / 8);
        const int64_t columns = g.total / ((int64_t)B.n * W);
        const unsigned blocks = (unsigned)(columns * B.strip_groups * B.chunks);
        if (!launch_box_strip(op == TM_MORPH_EROSION, pass[i].rh, pass[i].rv, B, blocks, s) || cudaGetLastError() != cudaSuccess) {
            rc = TM_EDT_ERR_CUDA;
            break;
        }
        ++launches;
        src = dst;
    }
    if (ws) cudaFreeAsync(ws, s);
    if (rc == TM_EDT_OK) tmedt::shared_record(-1, launches);
    return rc;
}

// Binary erosion / dilation on bit-packed lines (morph_bits.cuh) when the shape allows it; returns -1 when it does
// not, and the caller goes on with the byte kernels.
static int run_binary_bits(const Geometry& g, const std::vector<Entry>& entries, const uint8_t* input, uint8_t* output,
                           bool erosion, int border_value, cudaStream_t s) {
    const int nd = g.ndim, W = g.ext[nd - 1];
    const bool fast = W % 32 == 0 && !((uintptr_t)input & 31u) && !((uintptr_t)output & 31u);
    if (nd > 4 || (!fast && (W % 4 != 0 || W < 32 || ((uintptr_t)input & 3u) || ((uintptr_t)output & 3u)))) return -1;
    const int words_per_line = (W + 31) / 32;
    if ((g.total / W + 7) / 8 * ((words_per_line + 31) / 32) > (int64_t)INT32_MAX) return -1;  // blocks of the line kernel
    std::vector<LineGroup> groups;
    for (const Entry& en : entries) {
        const int dx = en.off[nd - 1];
        if (dx < -31 || dx > 31) return -1;
        LineGroup* grp = nullptr;
        for (LineGroup& c : groups) {
            bool same = true;
            for (int a = 0; a < nd - 1; ++a) same = same && c.off[a] == en.off[a];
            if (same) { grp = &c; break; }
        }
        if (!grp) {
            LineGroup n;
            memset(&n, 0, sizeof(n));
            for (int a = 0; a < nd - 1; ++a) { n.off[a] = en.off[a]; n.line_offset += (int64_t)en.off[a] * (g.stride[a] / W); }
            groups.push_back(n);
            grp = &groups.back();
        }
        grp->mask |= (uint64_t)1 << (dx + 31);
    }
    if ((int)groups.size() > kMaxLineGroups) return -1;
    // an element that reaches over the last two axes only: packing and combining in one kernel
    {
        bool last_two = true;
        int dy_lo = 0, dy_hi = 0;
        for (const LineGroup& c : groups) {
            for (int a = 0; a < nd - 2; ++a) last_two = last_two && c.off[a] == 0;
            if (nd >= 2) { dy_lo = std::min(dy_lo, (int)c.off[nd - 2]); dy_hi = std::max(dy_hi, (int)c.off[nd - 2]); }
        }
        const int64_t lines = g.total / W;
        const unsigned chunks = (unsigned)((words_per_line + 31) / 32);
        if (last_two && dy_lo >= -kFusedReach && dy_hi <= kFusedReach && (lines + 31) / 32 * chunks <= (int64_t)INT32_MAX) {
            BitsParams B;
            memset(&B, 0, sizeof(B));
            B.in = input; B.out = output;
            for (size_t i = 0; i < groups.size(); ++i) B.groups[i] = groups[i];
            B.n_groups = (int)groups.size();
            B.ndim = nd; B.words = words_per_line; B.lines = lines; B.lines_per_image = g.V / W; B.fast = fast;
            for (int a = 0; a < nd; ++a) B.ext[a] = g.ext[a];
            B.border_value = border_value ? 1 : 0;
            const unsigned blocks = (unsigned)((lines + 31) / 32) * chunks;
            const int H = nd >= 2 ? g.ext[nd - 2] : 1;
            if (fast) {
                if (erosion) binary_fused2d_kernel<true, true><<<blocks, 256, 0, s>>>(B, chunks, H, dy_lo, dy_hi);
                else binary_fused2d_kernel<false, true><<<blocks, 256, 0, s>>>(B, chunks, H, dy_lo, dy_hi);
            } else {
                if (erosion) binary_fused2d_kernel<true, false><<<blocks, 256, 0, s>>>(B, chunks, H, dy_lo, dy_hi);
                else binary_fused2d_kernel<false, false><<<blocks, 256, 0, s>>>(B, chunks, H, dy_lo, dy_hi);
            }
            const cudaError_t e = cudaGetLastError();
            if (e != cudaSuccess) { tmedt::shared_record((int)e, 0); return TM_EDT_ERR_CUDA; }
            tmedt::shared_record(-1, 1);
            return TM_EDT_OK;
        }
    }
    const int64_t words = g.total / W * words_per_line;
    char* dev = nullptr;
    cudaError_t e = tmedt::shared_scratch_alloc((void**)&dev, (size_t)words * 4, s);
    if (e != cudaSuccess) { cudaGetLastError(); tmedt::shared_record((int)e, 0); return TM_EDT_ERR_ALLOC; }
    {
        BitsParams B;
        memset(&B, 0, sizeof(B));
        B.in = input; B.out = output; B.bits = reinterpret_cast<uint32_t*>(dev);
        for (size_t i = 0; i < groups.size(); ++i) B.groups[i] = groups[i];
        B.n_groups = (int)groups.size();
        B.ndim = nd; B.words = words_per_line; B.lines = g.total / W; B.lines_per_image = g.V / W; B.fast = fast;
        for (int a = 0; a < nd; ++a) B.ext[a] = g.ext[a];
        B.border_value = border_value ? 1 : 0;
        const unsigned blocks = (unsigned)((words + 255) / 256);
        binary_pack_kernel<<<blocks, 256, 0, s>>>(B);
        const unsigned chunks = (unsigned)((B.words + 31) / 32);
        const int L = nd >= 2 && g.ext[nd - 2] % 4 == 0 ? 4 : 1;  // lines per lane
        const unsigned lblocks = (unsigned)((B.lines / L + 7) / 8) * chunks;
#define TM_BITS_LINES(LL, NDV)                                                                                 \
    do {                                                                                                       \
        if (erosion) binary_lines_kernel<true, LL, NDV><<<lblocks, dim3(32, 8), 0, s>>>(B, chunks);             \
        else binary_lines_kernel<false, LL, NDV><<<lblocks, dim3(32, 8), 0, s>>>(B, chunks);                    \
    } while (0)
        if (L == 4) { if (nd == 2) TM_BITS_LINES(4, 2); else if (nd == 3) TM_BITS_LINES(4, 3); else TM_BITS_LINES(4, 4); }
        else { if (nd == 1) TM_BITS_LINES(1, 1); else if (nd == 2) TM_BITS_LINES(1, 2); else if (nd == 3) TM_BITS_LINES(1, 3); else TM_BITS_LINES(1, 4); }
#undef TM_BITS_LINES
        e = cudaGetLastError();
    }
    cudaFreeAsync(dev, s);
    if (e != cudaSuccess) { tmedt::shared_record((int)e, 0); return TM_EDT_ERR_CUDA; }
    tmedt::shared_record(-1, 2);
    return TM_EDT_OK;
}

template <typename T, bool BINARY>
int run(const T* input, int ndim, const int64_t* shape, const uint8_t* fp, const float* st, const int64_t* fp_shape,
        const int64_t* origin, int op, int mode, float cval, int border_value, void* output, tm_edt_stream_t stream,
        bool allow_separable) {
    if (!input || !output) return TM_EDT_ERR_INVALID_ARG;
    if (op != TM_MORPH_EROSION && op != TM_MORPH_DILATION) return TM_EDT_ERR_INVALID_ARG;
    if (mode < TM_MORPH_CONSTANT || mode > TM_MORPH_WRAP) return TM_EDT_ERR_INVALID_ARG;
    Geometry g;
    int rc = check_geometry(ndim, shape, g);
    if (rc != TM_EDT_OK) return rc;
    std::vector<Entry> entries;
    Params P;
    memset(&P, 0, sizeof(P));
    rc = flatten(g, fp, st, fp_shape, origin, op == TM_MORPH_DILATION, entries, P.lo, P.hi);
    if (rc != TM_EDT_OK) return rc;
    if (g.total == 0) { tmedt::shared_record(-1, 0); return TM_EDT_OK; }
    const size_t out_bytes = (size_t)g.total * (BINARY ? 1 : 4);
    if (tmedt::shared_overlap(input, (size_t)g.total * sizeof(T), output, out_bytes)) return TM_EDT_ERR_INVALID_ARG;
    if (((uintptr_t)input % sizeof(T)) || ((uintptr_t)output % (BINARY ? 1 : 4))) return TM_EDT_ERR_INVALID_ARG;
    if (!tmedt::shared_is_device_ptr(input) || !tmedt::shared_is_device_ptr(output)) return TM_EDT_ERR_BAD_POINTER;
    if (g.total > (int64_t)INT32_MAX * 128) return TM_EDT_ERR_UNSUPPORTED;
    if (BINARY && allow_separable) {
        const int rb = run_binary_bits(g, entries, reinterpret_cast<const uint8_t*>(input), static_cast<uint8_t*>(output),
                                       op == TM_MORPH_EROSION, border_value, (cudaStream_t)stream);
        if (rb >= 0) return rb;
    }
    if (!BINARY && allow_separable) {
        int64_t box = 1;
        bool flat = true;
        for (int a = 0; a < ndim; ++a) box *= fp_shape[a];
        for (const Entry& en : entries) flat = flat && en.s == 0.0f;
        if (flat && (int64_t)entries.size() == box && box <= (int64_t)sizeof(uint8_t) * 256 * 9 && box > 1) {
            int64_t last2 = fp_shape[ndim - 1] * (ndim >= 2 ? fp_shape[ndim - 2] : 1);
            if (last2 <= 256 * 9) {
                const int rq = run_box_quads(reinterpret_cast<const float*>(input), ndim, fp_shape, origin, op, mode, cval,
                                             static_cast<float*>(output), stream, g);
                if (rq >= 0) return rq;
            }
        }
    }
    if (allow_separable && ndim >= 2 && entries.size() >= 20) {
        int64_t box = 1;
        bool flat = true;
        for (int a = 0; a < ndim; ++a) box *= fp_shape[a];
        for (const Entry& en : entries) flat = flat && en.s == 0.0f;
        if (flat && (int64_t)entries.size() == box)
            return run_box<T, BINARY>(input, ndim, shape, fp_shape, origin, op, mode, cval, border_value, output, stream,
                                      (size_t)g.total);
    }
    cudaStream_t s = (cudaStream_t)stream;
    int launches = 0;
    void* dev = nullptr;
    const size_t bytes = entries.size() * sizeof(Entry);
    cudaError_t e = tmedt::shared_scratch_alloc(&dev, bytes, s);
    if (e != cudaSuccess) { cudaGetLastError(); tmedt::shared_record((int)e, 0); return TM_EDT_ERR_ALLOC; }
    e = cudaMemcpyAsync(dev, entries.data(), bytes, cudaMemcpyHostToDevice, s);  // pageable source: consumed on return
    if (e == cudaSuccess) {
        P.in = input; P.out = output; P.entries = static_cast<const Entry*>(dev); P.n_entries = (int)entries.size();
        P.ndim = g.ndim; P.total = g.total; P.V = (int)g.V;
        for (int a = 0; a < g.ndim; ++a) { P.ext[a] = g.ext[a]; P.stride[a] = g.stride[a]; }
        for (int a = 0; a < g.ndim; ++a) { P.flat_lo += (int64_t)P.lo[a] * g.stride[a]; P.flat_hi += (int64_t)P.hi[a] * g.stride[a]; }
        P.mode = BINARY ? kConstant : mode;
        P.cval = cval; P.border_value = border_value ? 1 : 0;
        // eight or four voxels per lane (256 or 128 consecutive voxels of a row per warp) when rows are a multiple of that
        const int vpt = g.ext[g.ndim - 1] % 256 == 0 ? 8 : (g.ext[g.ndim - 1] % 128 == 0 ? 4 : 1);
        const int64_t threads = (g.total + vpt - 1) / vpt;
        const unsigned blocks = (unsigned)((threads + 255) / 256);
        const size_t smem = entries.size() * 8;
        const bool ero = op == TM_MORPH_EROSION;
        bool flat = true;
        for (const Entry& en : entries) flat = flat && en.s == 0.0f;
#define TM_MORPH_LAUNCH(V, F)                                                                                    \
    do {                                                                                                         \
        if (ero) morph_interior_kernel<T, true, BINARY, V, F><<<blocks, 256, smem, s>>>(P);                       \
        else morph_interior_kernel<T, false, BINARY, V, F><<<blocks, 256, smem, s>>>(P);                          \
    } while (0)
        if (BINARY || flat) { if (vpt == 8) TM_MORPH_LAUNCH(8, true); else if (vpt == 4) TM_MORPH_LAUNCH(4, true); else TM_MORPH_LAUNCH(1, true); }
        else { if (vpt == 8) TM_MORPH_LAUNCH(8, false); else if (vpt == 4) TM_MORPH_LAUNCH(4, false); else TM_MORPH_LAUNCH(1, false); }
#undef TM_MORPH_LAUNCH
        launches = 1;
        // border slabs: per axis the voxels that fail the interior test
        Slabs S;
        memset(&S, 0, sizeof(S));
        for (int a = 0; a < g.ndim; ++a) {
            const int n = g.ext[a], grp = 1;  // the interior kernel tests every voxel by itself
            const int low_w = std::min(n, ((std::max(0, -P.lo[a]) + grp - 1) / grp) * grp);       // [0, low_w)
            // first failing group start: the smallest multiple of grp with x0 + grp - 1 + hi >= n
            const int need = n - std::max(0, P.hi[a]) - (grp - 1);
            const int high_s = std::max(0, std::min(n, ((std::max(0, need) + grp - 1) / grp) * grp));  // [high_s, n)
            auto add = [&](int start, int width) {
                if (width <= 0) return;
                S.axis[S.count] = a; S.start[S.count] = start; S.width[S.count] = width;
                S.first[S.count + 1] = S.first[S.count] + g.V / n * width;
                ++S.count;
            };
            if (low_w >= high_s) add(0, n);  // the two slabs meet: the whole axis is border
            else { add(0, low_w); add(high_s, n - high_s); }
        }
        const int64_t items = g.images * S.first[S.count];
        if (items > 0) {
            if (items > (int64_t)INT32_MAX * 128) e = cudaErrorInvalidValue;
            else {
                const unsigned bb = (unsigned)((items + 255) / 256);
                if (ero) morph_border_kernel<T, true, BINARY><<<bb, 256, 0, s>>>(P, S, items);
                else morph_border_kernel<T, false, BINARY><<<bb, 256, 0, s>>>(P, S, items);
                launches = 2;
            }
        }
        if (e == cudaSuccess) e = cudaGetLastError();
    }
    cudaFreeAsync(dev, s);
    if (e != cudaSuccess) { tmedt::shared_record((int)e, 0); return TM_EDT_ERR_CUDA; }
    tmedt::shared_record(-1, launches);
    return TM_EDT_OK;
}

}  // namespace

extern "C" {

int tm_grey_morph(const float* input, int ndim, const int64_t* shape, const uint8_t* footprint, const float* structure,
                  const int64_t* fp_shape, const int64_t* origin, int op, int mode, float cval, float* output,
                  tm_edt_stream_t stream) {
    return run<float, false>(input, ndim, shape, footprint, structure, fp_shape, origin, op, mode, cval, 0, output, stream);
}

int tm_binary_morph(const uint8_t* input, int ndim, const int64_t* shape, const uint8_t* structure, const int64_t* fp_shape,
                    const int64_t* origin, int op, int border_value, uint8_t* output, tm_edt_stream_t stream) {
    return run<uint8_t, true>(input, ndim, shape, structure, nullptr, fp_shape, origin, op, TM_MORPH_CONSTANT, 0.0f,
                              border_value, output, stream);
}

}  // extern "C"
