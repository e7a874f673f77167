// Internal helpers of the CCL library: status/error text, descriptor validation and the
// address-map arithmetic (Eq. 1-3) shared by the host entry points and the kernels.
#pragma once

#include <cstdarg>
#include <cstdint>
#include <cstdio>

#include <cuda_runtime.h>

#include "ccl.h"

#if defined(__CUDACC__)
#define CCL_HD __host__ __device__ __forceinline__
#else
#define CCL_HD inline
#endif

namespace ccl {

ccl_status fail(ccl_status s, const char* fmt, ...);   // records the thread-local message, returns s
void clear_error();
void count_launch(int n = 1);                              // bookkeeping for ccl_launch_count()

#define CCL_CUDA_TRY(expr)                                                                      \
    do {                                                                                        \
        cudaError_t e__ = (expr);                                                               \
        if (e__ != cudaSuccess) return ::ccl::fail(CCL_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
    } while (0)

// Flattened view of a ccl_mat: everything a kernel needs to address it.
//   offset(r,c) = (r / h) * stride + (r % h) * w_row ... see map() below.
struct MatView {
    int64_t rows, cols;
    int64_t w;        // width of a strip row in elements (ceil(cols/P) for PART_COLS, else cols)
    int64_t h;        // rows per strip (ceil(rows/P) for PART_ROWS, else rows)
    int64_t wlast;    // width of the LAST strip's rows (= w unless cols is not a multiple of P)
    int64_t hlast;    // rows of the LAST strip (= h unless rows is not a multiple of P)
    int64_t last_span;// elements the last strip occupies, its alignment padding included
    int64_t stride;   // elements between strip bases (0 when there is a single strip)
    int64_t nstrips;  // P for CCL layouts, else 1
    int32_t e;        // element bytes
    int32_t split;    // 0 none, 1 rows, 2 cols (effective: 0 for row-major)
    int64_t ichunk;   // page-interleaved CCL: elements per chunk (0 = strips stored one after the other)
    int64_t ichunks;  // page-interleaved CCL: chunks per strip
};

// Page-interleaved CCL: element o of strip g's packed contents -> element offset in the buffer
// (chunk j of strip g is stored as chunk j*P + g).
CCL_HD int64_t interleave(const MatView& v, int64_t g, int64_t o) {
    int64_t j = o / v.ichunk;
    return (j * v.nstrips + g) * v.ichunk + (o - j * v.ichunk);
}

// Width of strip g's rows / rows of strip g: only the last strip of a dimension that P does not divide differs.
CCL_HD int64_t strip_w_of(const MatView& v, int64_t g) { return g == v.nstrips - 1 ? v.wlast : v.w; }
CCL_HD int64_t strip_h_of(const MatView& v, int64_t g) { return g == v.nstrips - 1 ? v.hlast : v.h; }
CCL_HD bool ragged(const MatView& v) { return v.wlast != v.w || v.hlast != v.h; }

CCL_HD int64_t map(const MatView& v, int64_t r, int64_t c) {
    if (v.split == 2) {                      // Eq. 1 + Eq. 3 (w = ceil(cols / P); a narrower last strip keeps its own row pitch)
        int64_t g = c / v.w, cp = c - g * v.w;
        const int64_t wg = strip_w_of(v, g);
        if (v.ichunk) return interleave(v, g, r * wg + cp);
        return g * v.stride + r * wg + cp;
    }
    if (v.split == 1) {                      // strips of h whole rows
        int64_t g = r / v.h, rp = r - g * v.h;
        if (v.ichunk) return interleave(v, g, rp * v.cols + c);
        return g * v.stride + rp * v.cols + c;
    }
    return r * v.cols + c;                   // Eq. 2
}

CCL_HD int64_t buffer_elems(const MatView& v) {
    if (v.ichunk) return v.ichunks * v.nstrips * v.ichunk;
    return v.split ? (v.nstrips - 1) * v.stride + v.last_span : v.rows * v.cols;
}

// Validates a descriptor and flattens it.  `what` names the argument in error messages.
ccl_status make_view(const ccl_mat* m, const char* what, MatView* out);

}  // namespace ccl
