// tm_cdt / tm_bfdt: host side (see include/tm_cdt.h and cdt.cuh).
#include <math.h>
#include <string.h>

#include "../../include/tm_cdt.h"
#include "cdt.cuh"
#include "host_shared.h"

namespace tmedt { cudaError_t launch_row_dist16(const uint8_t* mask, uint16_t* out, int64_t rows, int n0, cudaStream_t st); }

using namespace tmcdt;

namespace {

struct Geo { int ndim; int64_t images, V, total; int64_t ext[8]; };

int geometry(int ndim, const int64_t* shape, int max_ndim, Geo& g) {
    if (ndim < 1 || ndim > max_ndim || !shape) return TM_EDT_ERR_INVALID_ARG;
    if (shape[0] < 0 || shape[1] < 0) return TM_EDT_ERR_INVALID_ARG;
    g.ndim = ndim; g.images = shape[0] * shape[1]; g.V = 1;
    for (int a = 0; a < ndim; ++a) {
        if (shape[2 + a] < 0) return TM_EDT_ERR_INVALID_ARG;
        if (shape[2 + a] > 0 && g.V > (int64_t)INT32_MAX / shape[2 + a]) return TM_EDT_ERR_UNSUPPORTED;
        g.V *= shape[2 + a];
        g.ext[a] = shape[2 + a];
    }
    if (g.images > 0 && g.V > 0 && g.images > ((int64_t)1 << 40) / g.V) return TM_EDT_ERR_UNSUPPORTED;
    g.total = g.images * g.V;
    return TM_EDT_OK;
}

}  // namespace

namespace tmedt {

// Used by the Euclidean transform's two-axis path as well: the row distances are the same for every metric.
cudaError_t launch_row_dist16(const uint8_t* mask, uint16_t* out, int64_t rows, int n0, cudaStream_t st) {
    Row16Params R;
    R.mask = mask; R.out = out; R.rows = rows; R.n0 = n0; R.words = n0 / 32; R.edge = nullptr; R.nb = 0;
    const int64_t warps = (rows + 32 / R.words - 1) / (32 / R.words);
    cdt_row16_kernel<true><<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(R);
    return cudaGetLastError();
}

}  // namespace tmedt

extern "C" {

int tm_cdt(const uint8_t* input, int ndim, const int64_t* shape, int metric, int32_t* out_dist, tm_edt_stream_t stream) {
    if (!input || !out_dist) return TM_EDT_ERR_INVALID_ARG;
    if (metric != TM_METRIC_TAXICAB && metric != TM_METRIC_CHESSBOARD) return TM_EDT_ERR_INVALID_ARG;
    Geo g;
    int rc = geometry(ndim, shape, 8, g);
    if (rc != TM_EDT_OK) return rc;
    if (g.total == 0) { tmedt::shared_record(-1, 0); return TM_EDT_OK; }
    if ((uintptr_t)out_dist & 3u) return TM_EDT_ERR_INVALID_ARG;
    if (tmedt::shared_overlap(input, (size_t)g.total, out_dist, (size_t)g.total * 4)) return TM_EDT_ERR_INVALID_ARG;
    if (!tmedt::shared_is_device_ptr(input) || !tmedt::shared_is_device_ptr(out_dist)) return TM_EDT_ERR_BAD_POINTER;
    if (g.total > (int64_t)INT32_MAX * 128) return TM_EDT_ERR_UNSUPPORTED;
    // axes with more than one voxel, contiguous axis first; an image of one voxel keeps its last axis
    int axes[8], E = 0;
    for (int a = ndim - 1; a >= 0; --a)
        if (g.ext[a] > 1) axes[E++] = a;
    if (E == 0) axes[E++] = ndim - 1;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t buf = (((size_t)g.total * 4) + 255) & ~(size_t)255;
    // The first two axes on 16-bit values (cdt.cuh): rows of up to 1024 voxels, a multiple of 32 (or of 4 from 64 voxels
    // on: the last word of a row is then ragged and the 16-bit rows are padded to whole words), a second axis of up to
    // 1024 rows whose stride is the row length.
    bool fast = false;
    size_t fast_bytes = 0;
    if (E >= 2 && axes[0] == ndim - 1) {
        const int64_t n0 = g.ext[axes[0]], n1 = g.ext[axes[1]];
        const bool rows_ok = n0 % 32 == 0 ? ((uintptr_t)input & 31u) == 0 : (n0 % 4 == 0 && n0 >= 64 && ((uintptr_t)input & 3u) == 0);
        fast = rows_ok && n0 <= 1024 && n1 <= 1024 && ((uintptr_t)out_dist & 15u) == 0 && g.total / (32 * n1) <= (int64_t)INT32_MAX;
        if (fast) {
            const int64_t fpitch = (n0 + 31) / 32 * 32, rows = g.total / n0, slabs = rows / n1;
            const int64_t segs = (n1 + kSegRows - 1) / kSegRows, groups = (n0 + 127) / 128;
            fast_bytes = (size_t)rows * fpitch * 2 + (size_t)slabs * segs * fpitch * 2 + (size_t)slabs * (groups - 1) * 2 * n1 * 2 +
                         (size_t)rows * (groups - 1) * 4 + 1024;
            fast_bytes = (fast_bytes + 255) & ~(size_t)255;
        }
    }
    char* ws = nullptr;
    const size_t later = E > 2 ? 2 * buf : 0;  // the int32 images between the later passes
    if (E > 1) {
        cudaError_t e = tmedt::shared_scratch_alloc((void**)&ws, fast ? fast_bytes + later : (E > 2 ? 2 : 1) * buf, st);
        if (e != cudaSuccess) { cudaGetLastError(); tmedt::shared_record((int)e, 0); return TM_EDT_ERR_ALLOC; }
    }
    char* fast_ws = ws;
    char* tmp_base = fast ? ws + fast_bytes : ws;
    int32_t* tmp[2] = {reinterpret_cast<int32_t*>(tmp_base), reinterpret_cast<int32_t*>(tmp_base + buf)};
    const int32_t* prev = nullptr;
    cudaError_t e = cudaSuccess;
    const bool chess = metric == TM_METRIC_CHESSBOARD;
    int k0 = 0, launches_fast = 0;
    if (fast) {
        const int n0 = (int)g.ext[axes[0]], n1 = (int)g.ext[axes[1]];
        const int groups = (n0 + 127) / 128, words = (n0 + 31) / 32, fpitch = 32 * words;
        const int64_t slabs = g.total / ((int64_t)n1 * n0);
        const int segs = (n1 + kSegRows - 1) / kSegRows;
        // 16-bit values, pinned results and the gathered boundary columns
        uint16_t* f = reinterpret_cast<uint16_t*>(fast_ws);
        uint16_t* pd = f + (size_t)(g.total / n0) * fpitch;
        uint16_t* hd = pd + (size_t)slabs * segs * fpitch;
        uint16_t* edge = hd + (size_t)slabs * (groups - 1) * 2 * n1;
        Row16Params R;
        R.mask = input; R.out = f; R.rows = g.total / n0; R.n0 = n0; R.words = words;
        R.edge = chess && groups > 1 ? edge : nullptr; R.nb = groups - 1;
        const int64_t warps = (R.rows + 32 / R.words - 1) / (32 / R.words);
        if (n0 % 32 == 0) cdt_row16_kernel<true><<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(R);
        else cdt_row16_kernel<false><<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(R);
        SweepParams C;
        memset(&C, 0, sizeof(C));
        C.f = R.out; C.last = E == 2; C.out = C.last ? out_dist : tmp[1];
        C.slabs = slabs; C.inner = n0; C.n = n1; C.segs = segs; C.groups = groups; C.fpitch = fpitch;
        C.pd = pd; C.hd = hd; C.edge = edge;
        const int64_t row_blocks = (C.slabs * C.segs * (fpitch / 2) + 255) / 256;
        const int64_t col_blocks = chess ? C.slabs * (groups - 1) : 0;
        if (chess) cdt_pins_kernel<true><<<(unsigned)(row_blocks + col_blocks), 256, (size_t)n1 * 4, st>>>(C, (unsigned)row_blocks);
        else cdt_pins_kernel<false><<<(unsigned)row_blocks, 256, 0, st>>>(C, (unsigned)row_blocks);
        const int64_t pieces = C.slabs * C.segs * C.groups;
        if (chess) cdt_sweep_kernel<true><<<(unsigned)((pieces + 3) / 4), 128, 0, st>>>(C);
        else cdt_sweep_kernel<false><<<(unsigned)((pieces + 3) / 4), 128, 0, st>>>(C);
        launches_fast = 3;
        e = cudaGetLastError();
        prev = C.out;
        k0 = 2;
    }
    for (int k = k0; k < E && e == cudaSuccess; ++k) {
        PassParams P;
        memset(&P, 0, sizeof(P));
        P.mask = input; P.in = prev; P.total = g.total;
        P.first = k == 0; P.last = k == E - 1;
        P.out = P.last ? out_dist : tmp[k & 1];
        P.n = (int)g.ext[axes[k]];
        P.inner = 1;
        for (int a = axes[k] + 1; a < ndim; ++a) P.inner *= g.ext[a];
        if (k == 0 && P.inner == 1 && P.n <= 8192) {
            // contiguous lines: ballot words, same distance for both metrics
            RowParams R;
            R.mask = input; R.out = P.out; R.rows = g.total / P.n; R.n0 = P.n; R.last = P.last;
            cdt_row_kernel<<<(unsigned)((R.rows + 7) / 8), 256, 0, st>>>(R);
        } else if (k > 0 && P.n <= 1024) {
            // strided axis: (n x 32) strips in shared memory, (n x 16) for axes longer than 256 rows
            const int cw = P.n > 256 && P.inner >= 32 ? 16 : 32;
            const int strips = (int)((P.inner + cw - 1) / cw);
            const size_t smem = (size_t)P.n * cw * 4;
            auto kern = cw == 16 ? (chess ? cdt_strip_kernel<true, 16> : cdt_strip_kernel<false, 16>)
                                 : (chess ? cdt_strip_kernel<true, 32> : cdt_strip_kernel<false, 32>);
            if (smem > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            const int threads = P.n >= 384 ? (cw == 32 ? 512 : 256) : 256;
            kern<<<(unsigned)(g.total / ((int64_t)P.n * P.inner) * strips), threads, smem, st>>>(P, strips);
        } else {
            const unsigned blocks = (unsigned)((g.total + 255) / 256);
            if (chess) cdt_axis_kernel<true><<<blocks, 256, 0, st>>>(P);
            else cdt_axis_kernel<false><<<blocks, 256, 0, st>>>(P);
        }
        e = cudaGetLastError();
        prev = P.out;
    }
    if (ws) cudaFreeAsync(ws, st);
    if (e != cudaSuccess) { tmedt::shared_record((int)e, 0); return TM_EDT_ERR_CUDA; }
    tmedt::shared_record(-1, k0 ? launches_fast + E - 2 : E);
    return TM_EDT_OK;
}

int tm_bfdt(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling, int metric, float* out_dist,
            tm_edt_stream_t stream) {
    if (!input || !out_dist) return TM_EDT_ERR_INVALID_ARG;
    if (metric < TM_METRIC_EUCLIDEAN || metric > TM_METRIC_CHESSBOARD) return TM_EDT_ERR_INVALID_ARG;
    Geo g;
    int rc = geometry(ndim, shape, 4, g);
    if (rc != TM_EDT_OK) return rc == TM_EDT_ERR_INVALID_ARG && ndim > 4 && ndim <= 8 ? TM_EDT_ERR_UNSUPPORTED : rc;
    BruteParams P;
    memset(&P, 0, sizeof(P));
    for (int a = 0; a < ndim; ++a) {
        const double w = sampling ? sampling[a] : 1.0;
        if (!(w > 0.0) || !isfinite(w)) return TM_EDT_ERR_INVALID_ARG;
        P.w[a] = (float)w;
        P.ext[a] = (int)g.ext[a];
    }
    if (g.total == 0) { tmedt::shared_record(-1, 0); return TM_EDT_OK; }
    if (g.V > (1 << 24) || g.images > 65535) return TM_EDT_ERR_UNSUPPORTED;
    if ((uintptr_t)out_dist & 3u) return TM_EDT_ERR_INVALID_ARG;
    if (tmedt::shared_overlap(input, (size_t)g.total, out_dist, (size_t)g.total * 4)) return TM_EDT_ERR_INVALID_ARG;
    if (!tmedt::shared_is_device_ptr(input) || !tmedt::shared_is_device_ptr(out_dist)) return TM_EDT_ERR_BAD_POINTER;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t b_sites = (((size_t)g.total * 4) + 255) & ~(size_t)255, b_counts = (((size_t)g.images * 4) + 255) & ~(size_t)255;
    char* ws = nullptr;
    cudaError_t e = tmedt::shared_scratch_alloc((void**)&ws, b_sites + b_counts, st);
    if (e != cudaSuccess) { cudaGetLastError(); tmedt::shared_record((int)e, 0); return TM_EDT_ERR_ALLOC; }
    int32_t* sites = reinterpret_cast<int32_t*>(ws);
    int32_t* counts = reinterpret_cast<int32_t*>(ws + b_sites);
    e = cudaMemsetAsync(counts, 0, (size_t)g.images * 4, st);
    if (e == cudaSuccess) {
        collect_background_kernel<<<(unsigned)((g.total + 255) / 256), 256, 0, st>>>(input, sites, counts, g.total, (int)g.V);
        P.mask = input; P.sites = sites; P.counts = counts; P.out = out_dist; P.V = (int)g.V;
        const dim3 grid((unsigned)((g.V + 255) / 256), (unsigned)g.images);
#define TM_BRUTE(M, R) brute_kernel<M, R><<<grid, 256, 0, st>>>(P)
#define TM_BRUTE_RANK(M)                                                                              \
    do {                                                                                              \
        if (ndim == 1) TM_BRUTE(M, 1); else if (ndim == 2) TM_BRUTE(M, 2); else if (ndim == 3) TM_BRUTE(M, 3); else TM_BRUTE(M, 4); \
    } while (0)
        if (metric == TM_METRIC_EUCLIDEAN) TM_BRUTE_RANK(0);
        else if (metric == TM_METRIC_TAXICAB) TM_BRUTE_RANK(1);
        else TM_BRUTE_RANK(2);
#undef TM_BRUTE_RANK
#undef TM_BRUTE
        e = cudaGetLastError();
    }
    cudaFreeAsync(ws, st);
    if (e != cudaSuccess) { tmedt::shared_record((int)e, 0); return TM_EDT_ERR_CUDA; }
    tmedt::shared_record(-1, 2);
    return TM_EDT_OK;
}

}  // extern "C"
