// Host-only entry points: the address map (Eq. 1-3), sizes, error text.
#include <atomic>
#include <cstring>

#include "ccl_common.h"

namespace ccl {

static thread_local char g_err[512] = "";

ccl_status fail(ccl_status s, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return s;
}

void clear_error() { g_err[0] = 0; }

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }
uint64_t launches() { return g_launches.load(std::memory_order_relaxed); }

ccl_status make_view(const ccl_mat* m, const char* what, MatView* out) {
    if (!m) return fail(CCL_ERR_INVALID_ARG, "%s: NULL descriptor", what);
    if (m->rows <= 0 || m->cols <= 0) return fail(CCL_ERR_INVALID_ARG, "%s: rows and cols must be positive", what);
    if (m->elem_bytes != 1 && m->elem_bytes != 2 && m->elem_bytes != 4)
        return fail(CCL_ERR_INVALID_ARG, "%s: elem_bytes must be 1, 2 or 4", what);
    if (m->P < 1) return fail(CCL_ERR_INVALID_ARG, "%s: P must be >= 1", what);
    if (m->layout != CCL_ROWMAJOR && m->layout != CCL_CCL && m->layout != CCL_CCL_INTERLEAVED) return fail(CCL_ERR_INVALID_ARG, "%s: unknown layout", what);
    if (m->part != CCL_PART_NONE && m->part != CCL_PART_ROWS && m->part != CCL_PART_COLS)
        return fail(CCL_ERR_INVALID_ARG, "%s: unknown part", what);
    if (m->strip_align_bytes < 0 || m->strip_align_bytes % m->elem_bytes)
        return fail(CCL_ERR_INVALID_ARG, "%s: strip_align_bytes must be a non-negative multiple of elem_bytes", what);
    // keep every byte offset comfortably inside int64
    if (m->rows > (INT64_C(1) << 40) || m->cols > (INT64_C(1) << 40) ||
        (double)m->rows * (double)m->cols * m->elem_bytes > 9.0e17)
        return fail(CCL_ERR_INVALID_ARG, "%s: matrix too large", what);
    MatView v;
    v.rows = m->rows; v.cols = m->cols; v.e = m->elem_bytes;
    v.w = m->cols; v.h = m->rows; v.wlast = v.w; v.hlast = v.h; v.last_span = 0; v.stride = 0; v.nstrips = 1; v.split = 0; v.ichunk = 0; v.ichunks = 0;
    if (m->layout != CCL_ROWMAJOR && m->part != CCL_PART_NONE) {
        // Eq. 1 with w = N / G rounded up: when P does not divide the split dimension the last strip keeps what is left
        // (at least one column / row, else CCL_ERR_SHAPE)
        int64_t packed, packed_last;
        if (m->part == CCL_PART_COLS) {
            v.w = (m->cols + m->P - 1) / m->P; v.wlast = m->cols - (int64_t)(m->P - 1) * v.w;
            if (v.wlast <= 0) return fail(CCL_ERR_SHAPE, "%s: %lld columns cannot be cut into %d strips of %lld (a strip would be empty)", what, (long long)m->cols, m->P, (long long)v.w);
            packed = m->rows * v.w; packed_last = m->rows * v.wlast; v.split = 2;
        } else {
            v.h = (m->rows + m->P - 1) / m->P; v.hlast = m->rows - (int64_t)(m->P - 1) * v.h;
            if (v.hlast <= 0) return fail(CCL_ERR_SHAPE, "%s: %lld rows cannot be cut into %d strips of %lld (a strip would be empty)", what, (long long)m->rows, m->P, (long long)v.h);
            packed = v.h * m->cols; packed_last = v.hlast * m->cols; v.split = 1;
        }
        v.nstrips = m->P;
        if (m->layout == CCL_CCL_INTERLEAVED) {
            if (m->strip_align_bytes <= 0) return fail(CCL_ERR_INVALID_ARG, "%s: the interleaved layout needs strip_align_bytes (the chunk size) > 0", what);
            v.ichunk = m->strip_align_bytes / m->elem_bytes;
            v.ichunks = (packed + v.ichunk - 1) / v.ichunk;
            v.stride = packed;                 // strip-local extent; strips are not stored one after the other
            v.last_span = packed_last;
        } else if (m->strip_align_bytes) {
            int64_t a = m->strip_align_bytes;
            v.stride = (packed * m->elem_bytes + a - 1) / a * a / m->elem_bytes;
            v.last_span = (packed_last * m->elem_bytes + a - 1) / a * a / m->elem_bytes;
        } else {
            v.stride = packed; v.last_span = packed_last;
        }
    }
    *out = v;
    return CCL_OK;
}

}  // namespace ccl

using namespace ccl;

extern "C" {

ccl_status ccl_map_offset(const ccl_mat* m, int64_t r, int64_t c, int64_t* elem_off) {
    MatView v;
    ccl_status s = make_view(m, "ccl_map_offset", &v);
    if (s) return s;
    if (!elem_off) return fail(CCL_ERR_INVALID_ARG, "ccl_map_offset: NULL output");
    if (r < 0 || c < 0 || r >= v.rows || c >= v.cols) return fail(CCL_ERR_INVALID_ARG, "ccl_map_offset: (r,c) out of range");
    *elem_off = map(v, r, c);
    return CCL_OK;
}

ccl_status ccl_map_inverse(const ccl_mat* m, int64_t off, int64_t* r, int64_t* c) {
    MatView v;
    ccl_status s = make_view(m, "ccl_map_inverse", &v);
    if (s) return s;
    if (!r || !c) return fail(CCL_ERR_INVALID_ARG, "ccl_map_inverse: NULL output");
    if (off < 0 || off >= buffer_elems(v)) return fail(CCL_ERR_INVALID_ARG, "ccl_map_inverse: offset out of range");
    if (v.split == 0) { *r = off / v.cols; *c = off % v.cols; return CCL_OK; }
    int64_t g, rem;
    if (v.ichunk) {                        // undo the chunk interleave, then proceed as for a packed strip
        int64_t chunk = off / v.ichunk;
        g = chunk % v.nstrips;
        rem = (chunk / v.nstrips) * v.ichunk + off % v.ichunk;
    } else { g = off / v.stride; rem = off % v.stride; }
    const int64_t wg = strip_w_of(v, g), hg = strip_h_of(v, g);
    if (rem >= (v.split == 2 ? v.rows * wg : hg * v.cols)) return fail(CCL_ERR_PADDING, "ccl_map_inverse: offset lies in the padding of strip %lld", (long long)g);
    if (v.split == 2) { *r = rem / wg; *c = g * v.w + rem % wg; }
    else { *r = g * v.h + rem / v.cols; *c = rem % v.cols; }
    return CCL_OK;
}

ccl_status ccl_buffer_bytes(const ccl_mat* m, int64_t* bytes) {
    MatView v;
    ccl_status s = make_view(m, "ccl_buffer_bytes", &v);
    if (s) return s;
    if (!bytes) return fail(CCL_ERR_INVALID_ARG, "ccl_buffer_bytes: NULL output");
    *bytes = buffer_elems(v) * v.e;
    return CCL_OK;
}

ccl_status ccl_strip_stride(const ccl_mat* m, int64_t* elems) {
    MatView v;
    ccl_status s = make_view(m, "ccl_strip_stride", &v);
    if (s) return s;
    if (!elems) return fail(CCL_ERR_INVALID_ARG, "ccl_strip_stride: NULL output");
    if (v.split == 0) return fail(CCL_ERR_INVALID_ARG, "ccl_strip_stride: not a CCL layout");
    if (v.ichunk) return fail(CCL_ERR_INVALID_ARG, "ccl_strip_stride: not defined for the interleaved layout");
    *elems = v.stride;
    return CCL_OK;
}

const char* ccl_last_error(void) { return g_err; }
uint64_t ccl_launch_count(void) { return ccl::launches(); }
const char* ccl_version(void) { return "0.1"; }

}  // extern "C"
