// Chiplet-Contiguous Layout (CCL) -- CPU oracle.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct
// statement of what the CUDA library computes.  It shares no code, header,
// table or helper with the CUDA path and is never called by the product path;
// only the test-suite, the smoke check and the benchmark's CPU-baseline leg
// load it.
//
// Every function cites the passage of the paper it restates:
//   Eq. 1  : g = floor(n / w), n' = n mod w, w = N / G
//            (reading for N not a multiple of G, which the paper leaves out: w = ceil(N / G), Eq. 1 unchanged, the
//            last strip is narrower -- N - (G-1)*w columns, at least one -- and every strip stays a contiguous
//            rows x width block, strip g starting g strides in: a packed buffer is still a bijection onto [0, K*N))
//   Eq. 2  : index_row(k, n) = k*N + n
//   Eq. 3  : index_CCL(k, n) = g*K*w + k*w + n'
//   Sec. 3.2 (last paragraph): a strip of K*w elements may be aligned to the
//            placement granularity (strip_align_bytes below)
//   Sec. 2.2: C = A*B, one CTA per output tile streaming A and B along K;
//            a column region of a column-major operand is already contiguous
//            (PART_ROWS below)
//   Sec. 3.3 / 4.1 (the evaluated setting: plain 4 KB round-robin over address bits already gives the locality): the
//            page-interleaved variant of CCL (layout ORC_CCL_INTERLEAVED): strip g's j-th chunk of
//            strip_align_bytes is stored at chunk j*G + g, so an address-driven "chunk mod G" mapping
//            sends every strip to its own chiplet
//   Sec. 4.1: page-granularity placement policies (round-robin interleave,
//            coarse G-block placement) and the remote-traffic metric, here
//            WITHOUT the L2 filter: every byte a CTA touches is counted.
//
// Pinning status (tests/test_oracle_*.py, no GPU needed):
//   map / inverse : pinned (bijection, stride form of Sec. 3.3, Fig. 4(a)
//                   worked example, reshape/permute, slice sizes of Sec. 2.2)
//   repack        : pinned (permutation, round trip, strided-slice copies); the transposing form lives in
//                   oracle/__init__.py (repack_transposed, written from the map; pinned by the Fig. 4(a) example)
//   gemm          : pinned (identity, all-ones, library matmul, fp64 bound)
//   gemm_axpby    : pinned (alpha = 1, beta = 0 is gemm; alpha = 0, beta = 1 returns C; exact small integers)
//   gemm_swiglu   : pinned (gate/up pairing enumerated by hand, silu closed forms, numpy in float64)
//   traffic_lru   : the finite-L2 model (one CTA after the other, or waves in lockstep through K) is this file's own
//                   reading of Sec. 4.1; pinned by its limits (one-line cache =
//                   uncached count in whole lines, unbounded cache = ideal-L2 count, monotone in the ways) and a
//                   hand-run example; against the paper's Fig. 6 numbers it is PARITY UNPINNED (unreleased simulator)
//   traffic       : pinned by invariants, closed forms and a hand-enumerated
//                   tiny case; against the paper's Fig. 6 ratios it is
//                   PARITY UNPINNED (they need the unreleased L2 simulator).
//
// Build: g++ -O2 -std=c++17 -shared -fPIC -pthread (see oracle/build.py).

#include <cstdint>
#include <cstring>
#include <cstdlib>
#include <cmath>
#include <vector>
#include <thread>
#include <algorithm>

extern "C" {

enum { ORC_ROWMAJOR = 0, ORC_CCL = 1, ORC_CCL_INTERLEAVED = 2 };
enum { ORC_PART_NONE = 0, ORC_PART_ROWS = 1, ORC_PART_COLS = 2 };
enum { ORC_PLACE_RR = 0, ORC_PLACE_BLOCK = 1, ORC_PLACE_BEST = 2 };
enum { ORC_ASSIGN_N = 0, ORC_ASSIGN_M = 1, ORC_ASSIGN_EXPLICIT = 2, ORC_ASSIGN_2D = 3 };

// A stored matrix: rows x cols, cols contiguous in the row-major view.
typedef struct {
    int64_t rows, cols;
    int32_t elem_bytes;
    int32_t P;                  // the paper's G
    int32_t part;               // which stored dimension is split over chiplets
    int32_t layout;             // physical order of the buffer
    int64_t strip_align_bytes;  // ORC_CCL: 0 = packed (Eq. 3 literally), else strip bases rounded up to it;
                                // ORC_CCL_INTERLEAVED: the chunk size (required)
} orc_mat;

typedef struct {
    int64_t M, N, K;
    int32_t BM, BN;
    orc_mat A, B, C;
    int32_t a_trans, b_trans;
    int32_t P;
    int64_t page_bytes;
    int32_t place[3];
    int32_t assign;
    int32_t strip_tiling;
    int32_t part_m;             // ORC_ASSIGN_2D: the output is cut into part_m x (P / part_m) blocks, one per chiplet
} orc_traffic_desc;

}  // extern "C"

namespace {

bool mat_ok(const orc_mat& m) {
    if (m.rows <= 0 || m.cols <= 0 || m.P < 1) return false;
    if (m.elem_bytes != 1 && m.elem_bytes != 2 && m.elem_bytes != 4) return false;
    if (m.layout != ORC_ROWMAJOR && m.layout != ORC_CCL && m.layout != ORC_CCL_INTERLEAVED) return false;
    if (m.part < 0 || m.part > 2) return false;
    if (m.strip_align_bytes < 0 || m.strip_align_bytes % m.elem_bytes) return false;
    if (m.layout != ORC_ROWMAJOR) {                    // every strip holds at least one column / row
        if (m.part == ORC_PART_COLS && (int64_t)(m.P - 1) * ((m.cols + m.P - 1) / m.P) >= m.cols) return false;
        if (m.part == ORC_PART_ROWS && (int64_t)(m.P - 1) * ((m.rows + m.P - 1) / m.P) >= m.rows) return false;
    }
    if (m.layout == ORC_CCL_INTERLEAVED && m.part != ORC_PART_NONE && m.strip_align_bytes <= 0) return false;
    return true;
}

bool is_ccl(const orc_mat& m) { return m.layout != ORC_ROWMAJOR && m.part != ORC_PART_NONE; }
bool is_interleaved(const orc_mat& m) { return m.layout == ORC_CCL_INTERLEAVED && m.part != ORC_PART_NONE; }

// Per-chiplet width w of Eq. 1 (split along columns) / rows per strip (split along rows): N / G, rounded up when N is
// not a multiple of G; the last strip then holds what is left.
int64_t strip_w(const orc_mat& m) { return (m.cols + m.P - 1) / m.P; }
int64_t strip_h(const orc_mat& m) { return (m.rows + m.P - 1) / m.P; }
int64_t strip_w_of(const orc_mat& m, int64_t g) { return std::min(strip_w(m), m.cols - g * strip_w(m)); }
int64_t strip_h_of(const orc_mat& m, int64_t g) { return std::min(strip_h(m), m.rows - g * strip_h(m)); }

// Elements of strip g, and of the largest strip (K*w in the paper's notation).
int64_t strip_elems_of(const orc_mat& m, int64_t g) {
    return (m.part == ORC_PART_COLS) ? m.rows * strip_w_of(m, g) : strip_h_of(m, g) * m.cols;
}
int64_t strip_elems(const orc_mat& m) { return strip_elems_of(m, 0); }
// Interleaved layout: chunks of strip_align_bytes each strip gets (those of the largest strip).
int64_t strip_chunks(const orc_mat& m) {
    return (strip_elems(m) * m.elem_bytes + m.strip_align_bytes - 1) / m.strip_align_bytes;
}

// Elements between the bases of two consecutive strips.  Packed: K*w (Eq. 3);
// aligned: K*w*e rounded up to the alignment (Sec. 3.2, last paragraph).
int64_t strip_stride(const orc_mat& m) {
    int64_t packed = strip_elems(m);
    if (m.strip_align_bytes == 0) return packed;
    int64_t bytes = packed * m.elem_bytes;
    int64_t up = (bytes + m.strip_align_bytes - 1) / m.strip_align_bytes * m.strip_align_bytes;
    return up / m.elem_bytes;
}

int64_t buffer_elems(const orc_mat& m) {
    if (!is_ccl(m)) return m.rows * m.cols;
    if (is_interleaved(m)) return strip_chunks(m) * m.P * (m.strip_align_bytes / m.elem_bytes);
    // P-1 strides, then the last strip (rounded up like the others when strips are aligned)
    int64_t last = strip_elems_of(m, m.P - 1);
    if (m.strip_align_bytes) last = (last * m.elem_bytes + m.strip_align_bytes - 1) / m.strip_align_bytes * m.strip_align_bytes / m.elem_bytes;
    return (int64_t)(m.P - 1) * strip_stride(m) + last;
}

// Interleaved layout: element `o` of strip g's packed contents (Eq. 3 inside the strip) lives in that strip's chunk
// j = o*e / S, which is stored as chunk j*G + g of the buffer.
int64_t interleave(const orc_mat& m, int64_t g, int64_t o) {
    int64_t S = m.strip_align_bytes, b = o * m.elem_bytes;
    return ((b / S * m.P + g) * S + b % S) / m.elem_bytes;
}

// Eq. 2 (row-major) or Eq. 1 + Eq. 3 (CCL) applied to stored coordinates.
int64_t map_offset(const orc_mat& m, int64_t r, int64_t c) {
    if (!is_ccl(m)) return r * m.cols + c;            // Eq. 2
    if (m.part == ORC_PART_COLS) {
        int64_t w = strip_w(m);                        // per-chiplet width
        int64_t g = c / w;                             // Eq. 1
        int64_t cp = c % w;                            // Eq. 1
        int64_t wg = strip_w_of(m, g);                 // = w, except in a narrower last strip
        if (is_interleaved(m)) return interleave(m, g, r * wg + cp);
        return g * strip_stride(m) + r * wg + cp;      // Eq. 3
    }
    // Split along rows: each strip is h whole rows, already contiguous (Sec. 2.2).
    int64_t h = strip_h(m);
    if (is_interleaved(m)) return interleave(m, r / h, (r % h) * m.cols + c);
    return (r / h) * strip_stride(m) + (r % h) * m.cols + c;
}

int map_inverse(const orc_mat& m, int64_t off, int64_t* r, int64_t* c) {
    if (off < 0 || off >= buffer_elems(m)) return -1;
    if (!is_ccl(m)) { *r = off / m.cols; *c = off % m.cols; return 0; }
    int64_t g, rem;
    if (is_interleaved(m)) {                           // undo the chunk interleave, then proceed as for a packed strip
        int64_t S = m.strip_align_bytes, b = off * m.elem_bytes, chunk = b / S;
        g = chunk % m.P;
        rem = (chunk / m.P * S + b % S) / m.elem_bytes;
    } else {
        int64_t st = strip_stride(m);
        g = off / st; rem = off % st;
    }
    if (rem >= strip_elems_of(m, g)) return -2;        // inside the padding of strip g
    if (m.part == ORC_PART_COLS) {
        int64_t wg = strip_w_of(m, g);
        *r = rem / wg; *c = g * strip_w(m) + rem % wg; return 0;
    }
    *r = g * strip_h(m) + rem / m.cols; *c = rem % m.cols; return 0;
}

inline float bf16_to_f32(uint16_t h) { uint32_t u = (uint32_t)h << 16; float f; std::memcpy(&f, &u, 4); return f; }
inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u; std::memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u);                   // round to nearest, ties to even (finite inputs)
    return (uint16_t)(u >> 16);
}

// ---- tile grid of the execution model (Sec. 2.2 / Sec. 4.1: one CTA per output tile) ----
struct Seg { int64_t lo, hi; };

// Tiles of one dimension cut into P strips of ceil(len/P) (the last one holds the rest).  strip_tiled: every strip is
// tiled on its own, so that no tile straddles two strips; otherwise plain ceil(len/B) tiles.
std::vector<Seg> tile_dim(int64_t len, int64_t B, int P, bool strip_tiled) {
    std::vector<Seg> v;
    if (!strip_tiled) { for (int64_t s = 0; s < len; s += B) v.push_back({s, std::min(len, s + B)}); return v; }
    int64_t w = (len + P - 1) / P;
    for (int g = 0; g < P; ++g) {
        const int64_t wg = std::min(w, len - g * w);
        for (int64_t s = 0; s < wg; s += B) v.push_back({g * w + s, g * w + std::min(wg, s + B)});
    }
    return v;
}

struct Tile { int64_t m0, m1, n0, n1; int32_t q; };

// every strip of a dimension of length len cut into P holds at least one element
bool strips_ok(int64_t len, int64_t P) { return P >= 1 && (P - 1) * ((len + P - 1) / P) < len; }

// Sec. 3.1 / 4.1: the output is partitioned over the chiplets and a CTA runs on the chiplet that owns its tile.
// N strips, M strips, an explicit table, or a 2-D partition into part_m x (P / part_m) blocks (chiplet qm * Pn + qn
// owns block (qm, qn)) -- Sec. 4.1 sweeps the output partition and keeps the best.
int enumerate_tiles(const orc_traffic_desc& d, const int32_t* explicit_q, std::vector<Tile>& out) {
    if (d.M <= 0 || d.N <= 0 || d.K <= 0 || d.BM <= 0 || d.BN <= 0 || d.P < 1) return -1;
    if (d.assign < 0 || d.assign > 3) return -1;
    int Pm = 1, Pn = 1;
    if (d.assign == ORC_ASSIGN_N) Pn = d.P;
    else if (d.assign == ORC_ASSIGN_M) Pm = d.P;
    else if (d.assign == ORC_ASSIGN_2D) {
        if (d.part_m < 1 || d.P % d.part_m) return -1;
        Pm = d.part_m; Pn = d.P / d.part_m;
    }
    if (!strips_ok(d.N, Pn) || !strips_ok(d.M, Pm)) return -1;
    if (d.assign == ORC_ASSIGN_EXPLICIT && !explicit_q) return -1;
    const int64_t wM = (d.M + Pm - 1) / Pm, wN = (d.N + Pn - 1) / Pn;
    auto tm = tile_dim(d.M, d.BM, Pm, Pm > 1 && d.strip_tiling);
    auto tn = tile_dim(d.N, d.BN, Pn, Pn > 1 && d.strip_tiling);
    for (size_t i = 0; i < tm.size(); ++i)
        for (size_t j = 0; j < tn.size(); ++j) {
            Tile t{tm[i].lo, tm[i].hi, tn[j].lo, tn[j].hi, 0};
            int64_t idx = (int64_t)i * (int64_t)tn.size() + (int64_t)j;
            if (d.assign == ORC_ASSIGN_EXPLICIT) { t.q = explicit_q[idx]; if (t.q < 0 || t.q >= d.P) return -1; }
            else t.q = (int32_t)((t.m0 / wM) * Pn + t.n0 / wN);      // the block holding the tile's first element
            out.push_back(t);
        }
    return 0;
}

// Stored-coordinate rectangle an output tile touches in operand X (0=A, 1=B, 2=C).
void tile_rect(const orc_traffic_desc& d, const Tile& t, int X, int64_t& r0, int64_t& r1, int64_t& c0, int64_t& c1) {
    if (X == 0) { if (!d.a_trans) { r0 = t.m0; r1 = t.m1; c0 = 0; c1 = d.K; } else { r0 = 0; r1 = d.K; c0 = t.m0; c1 = t.m1; } }
    else if (X == 1) { if (!d.b_trans) { r0 = 0; r1 = d.K; c0 = t.n0; c1 = t.n1; } else { r0 = t.n0; r1 = t.n1; c0 = 0; c1 = d.K; } }
    else { r0 = t.m0; r1 = t.m1; c0 = t.n0; c1 = t.n1; }
}

bool traffic_desc_ok(const orc_traffic_desc& d) {
    if (!mat_ok(d.A) || !mat_ok(d.B) || !mat_ok(d.C)) return false;
    if (d.page_bytes <= 0) return false;
    const orc_mat* ms[3] = {&d.A, &d.B, &d.C};
    for (int X = 0; X < 3; ++X) {
        if (d.page_bytes % ms[X]->elem_bytes) return false;
        if (d.place[X] < 0 || d.place[X] > 2) return false;
    }
    int64_t ar = d.a_trans ? d.K : d.M, ac = d.a_trans ? d.M : d.K;
    int64_t br = d.b_trans ? d.N : d.K, bc = d.b_trans ? d.K : d.N;
    return d.A.rows == ar && d.A.cols == ac && d.B.rows == br && d.B.cols == bc && d.C.rows == d.M && d.C.cols == d.N;
}

int64_t pages_of(const orc_mat& m, int64_t S) { return (buffer_elems(m) * m.elem_bytes + S - 1) / S; }

// Owner of a page under the fixed (address-driven) policies of Sec. 4.1.
//   RR   : consecutive fixed-size regions go to chiplets in address order.
//   BLOCK: the buffer is cut into P equal contiguous address blocks (coarse
//          placement); a page belongs to the block that holds its first byte.
int32_t fixed_owner(int place, int64_t page, int64_t S, int P, int64_t bytes_total) {
    if (place == ORC_PLACE_RR) return (int32_t)(page % P);
    int64_t o = (page * S * P) / bytes_total;
    return (int32_t)std::min<int64_t>(P - 1, o);
}

struct Visit { int64_t byte, len; };   // a contiguous piece inside one page

template <class F>
void for_each_piece_elem(const orc_traffic_desc& d, const orc_mat& m, int64_t r0, int64_t r1, int64_t c0, int64_t c1, F&& f) {
    for (int64_t r = r0; r < r1; ++r)
        for (int64_t c = c0; c < c1; ++c) f(map_offset(m, r, c) * m.elem_bytes, (int64_t)m.elem_bytes);
    (void)d;
}

// Run level: a stored row of the rectangle is contiguous inside one strip; cut it
// at strip boundaries (PART_COLS) and then at page boundaries.
template <class F>
void for_each_piece_run(const orc_traffic_desc& d, const orc_mat& m, int64_t r0, int64_t r1, int64_t c0, int64_t c1, F&& f) {
    int64_t S = d.page_bytes, e = m.elem_bytes;
    int64_t w = (is_ccl(m) && m.part == ORC_PART_COLS) ? strip_w(m) : m.cols;
    for (int64_t r = r0; r < r1; ++r) {
        int64_t c = c0;
        while (c < c1) {
            int64_t cend = std::min(c1, (c / w + 1) * w);
            if (is_interleaved(m)) {                   // contiguity also ends at every chunk of the interleave
                int64_t Si = m.strip_align_bytes;
                int64_t rr = (m.part == ORC_PART_ROWS) ? r % strip_h(m) : r;
                int64_t roww = (m.part == ORC_PART_COLS) ? strip_w_of(m, c / w) : m.cols;
                int64_t packed = (rr * roww + (m.part == ORC_PART_COLS ? c % w : c)) * e;   // byte inside the strip
                int64_t sub = std::min<int64_t>((cend - c) * e, (packed / Si + 1) * Si - packed);
                cend = c + sub / e;
            }
            int64_t b = map_offset(m, r, c) * e, bend = b + (cend - c) * e;
            while (b < bend) {
                int64_t pend = std::min(bend, (b / S + 1) * S);
                f(b, pend - b);
                b = pend;
            }
            c = cend;
        }
    }
}

template <bool RUNS>
int traffic_impl(const orc_traffic_desc& d, const int32_t* explicit_q, uint64_t* per_cta, uint64_t* const* per_page_out,
                 uint8_t* const* owner_out, uint64_t* totals) {
    if (!traffic_desc_ok(d)) return -1;
    std::vector<Tile> tiles;
    if (enumerate_tiles(d, explicit_q, tiles)) return -1;
    const orc_mat* ms[3] = {&d.A, &d.B, &d.C};
    int64_t S = d.page_bytes;
    int P = d.P;
    std::vector<uint64_t> hist[3];
    std::vector<uint8_t> own[3];
    for (int X = 0; X < 3; ++X) { hist[X].assign((size_t)pages_of(*ms[X], S) * P, 0); own[X].assign((size_t)pages_of(*ms[X], S), 0); }
    // pass 1: bytes of every page demanded by every chiplet
    for (const Tile& t : tiles)
        for (int X = 0; X < 3; ++X) {
            int64_t r0, r1, c0, c1; tile_rect(d, t, X, r0, r1, c0, c1);
            auto add = [&](int64_t byte, int64_t len) { hist[X][(size_t)(byte / S) * P + t.q] += (uint64_t)len; };
            if (RUNS) for_each_piece_run(d, *ms[X], r0, r1, c0, c1, add); else for_each_piece_elem(d, *ms[X], r0, r1, c0, c1, add);
        }
    // owner of every page
    for (int X = 0; X < 3; ++X) {
        int64_t np = pages_of(*ms[X], S), bytes_total = buffer_elems(*ms[X]) * ms[X]->elem_bytes;
        for (int64_t p = 0; p < np; ++p) {
            if (d.place[X] == ORC_PLACE_BEST) {        // best any page-granular mapping can do: the largest demander
                int best = 0;
                for (int q = 1; q < P; ++q) if (hist[X][(size_t)p * P + q] > hist[X][(size_t)p * P + best]) best = q;
                own[X][p] = (uint8_t)best;
            } else own[X][p] = (uint8_t)fixed_owner(d.place[X], p, S, P, bytes_total);
        }
    }
    // pass 2: classify every touched byte as local or remote
    for (int i = 0; i < 6; ++i) totals[i] = 0;
    for (size_t ti = 0; ti < tiles.size(); ++ti) {
        const Tile& t = tiles[ti];
        for (int X = 0; X < 3; ++X) {
            uint64_t loc = 0, rem = 0;
            int64_t r0, r1, c0, c1; tile_rect(d, t, X, r0, r1, c0, c1);
            auto cls = [&](int64_t byte, int64_t len) { if (own[X][(size_t)(byte / S)] == t.q) loc += (uint64_t)len; else rem += (uint64_t)len; };
            if (RUNS) for_each_piece_run(d, *ms[X], r0, r1, c0, c1, cls); else for_each_piece_elem(d, *ms[X], r0, r1, c0, c1, cls);
            per_cta[ti * 6 + X * 2 + 0] = loc; per_cta[ti * 6 + X * 2 + 1] = rem;
            totals[X * 2 + 0] += loc; totals[X * 2 + 1] += rem;
        }
    }
    for (int X = 0; X < 3; ++X) {
        if (per_page_out && per_page_out[X]) std::memcpy(per_page_out[X], hist[X].data(), hist[X].size() * 8);
        if (owner_out && owner_out[X]) std::memcpy(owner_out[X], own[X].data(), own[X].size());
    }
    return 0;
}

}  // namespace

extern "C" {

int orc_mat_valid(const orc_mat* m) { return mat_ok(*m) ? 1 : 0; }

// Eq. 1-3.  Returns 0 and the element offset, or -1 on a bad descriptor / coordinate.
int orc_map_offset(const orc_mat* m, int64_t r, int64_t c, int64_t* off) {
    if (!mat_ok(*m) || r < 0 || c < 0 || r >= m->rows || c >= m->cols) return -1;
    *off = map_offset(*m, r, c); return 0;
}

// Inverse of Eq. 3.  -2 when the offset falls into alignment padding.
int orc_map_inverse(const orc_mat* m, int64_t off, int64_t* r, int64_t* c) {
    if (!mat_ok(*m)) return -1;
    return map_inverse(*m, off, r, c);
}

int orc_strip_stride(const orc_mat* m, int64_t* elems) { if (!mat_ok(*m) || !is_ccl(*m) || is_interleaved(*m)) return -1; *elems = strip_stride(*m); return 0; }
int orc_buffer_bytes(const orc_mat* m, int64_t* bytes) { if (!mat_ok(*m)) return -1; *bytes = buffer_elems(*m) * m->elem_bytes; return 0; }

// Whole map as a table: out[r*cols + c] = offset (for bijection / stride-form pins).
int orc_map_table(const orc_mat* m, int64_t* out) {
    if (!mat_ok(*m)) return -1;
    for (int64_t r = 0; r < m->rows; ++r) for (int64_t c = 0; c < m->cols; ++c) out[r * m->cols + c] = map_offset(*m, r, c);
    return 0;
}

// Repack (Sec. 3.3: operands "adopt CCL" by a permutation copy).
// dir 0: dst[map(r,c)] = src[r*C + c], padding bytes = 0.  dir 1: dst[r*C + c] = src[map(r,c)].
int orc_repack(const orc_mat* m, const void* src, void* dst, int dir) {
    if (!mat_ok(*m)) return -1;
    int64_t e = m->elem_bytes;
    const uint8_t* s = (const uint8_t*)src; uint8_t* d = (uint8_t*)dst;
    if (dir == 0) std::memset(d, 0, (size_t)(buffer_elems(*m) * e));
    for (int64_t r = 0; r < m->rows; ++r)
        for (int64_t c = 0; c < m->cols; ++c) {
            int64_t lin = (r * m->cols + c) * e, off = map_offset(*m, r, c) * e;
            if (dir == 0) std::memcpy(d + off, s + lin, (size_t)e); else std::memcpy(d + lin, s + off, (size_t)e);
        }
    return 0;
}

// GEMM of Sec. 2.2, C = A*B, from the LOGICAL operands (never from CCL buffers):
//   ref32[m][n] = sum_k float(A[m][k]) * float(B[k][n]), k ascending, fp32 accumulate
//   ref64       = the same sum in double (bounds the fp32 oracle's own error)
//   out_bf16    = ref32 rounded to bf16, nearest-even
// A is stored row-major [M x K] (a_trans = 0) or [K x M] (a_trans = 1);
// B is stored row-major [K x N] (b_trans = 0) or [N x K] (b_trans = 1).
// Only the block rows [m0,m1) x cols [n0,n1) is produced, densely packed.
int orc_gemm(int64_t M, int64_t N, int64_t K, const uint16_t* A, int a_trans, const uint16_t* B, int b_trans,
             int64_t m0, int64_t m1, int64_t n0, int64_t n1, float* ref32, double* ref64, uint16_t* out_bf16, int threads) {
    if (M <= 0 || N <= 0 || K <= 0 || m0 < 0 || n0 < 0 || m1 > M || n1 > N || m0 >= m1 || n0 >= n1) return -1;
    int64_t nb = n1 - n0, mb = m1 - m0;
    // gather the needed columns of B as floats, [K x nb] (pure data movement)
    std::vector<float> Bf((size_t)(K * nb));
    for (int64_t k = 0; k < K; ++k)
        for (int64_t j = 0; j < nb; ++j)
            Bf[(size_t)(k * nb + j)] = bf16_to_f32(b_trans ? B[(n0 + j) * K + k] : B[k * N + n0 + j]);
    if (threads < 1) threads = 1;
    threads = (int)std::min<int64_t>(threads, mb);
    auto work = [&](int64_t lo, int64_t hi) {
        std::vector<float> acc((size_t)nb);
        std::vector<double> acc64(ref64 ? (size_t)nb : 0);
        for (int64_t i = lo; i < hi; ++i) {
            std::fill(acc.begin(), acc.end(), 0.0f);
            std::fill(acc64.begin(), acc64.end(), 0.0);
            for (int64_t k = 0; k < K; ++k) {
                float a = bf16_to_f32(a_trans ? A[k * M + (m0 + i)] : A[(m0 + i) * K + k]);
                const float* brow = &Bf[(size_t)(k * nb)];
                for (int64_t j = 0; j < nb; ++j) acc[(size_t)j] += a * brow[j];
                if (ref64) for (int64_t j = 0; j < nb; ++j) acc64[(size_t)j] += (double)a * (double)brow[j];
            }
            for (int64_t j = 0; j < nb; ++j) {
                if (ref32) ref32[i * nb + j] = acc[(size_t)j];
                if (ref64) ref64[i * nb + j] = acc64[(size_t)j];
                if (out_bf16) out_bf16[i * nb + j] = f32_to_bf16_rne(acc[(size_t)j]);
            }
        }
    };
    std::vector<std::thread> pool;
    int64_t per = (mb + threads - 1) / threads;
    for (int t = 0; t < threads; ++t) {
        int64_t lo = t * per, hi = std::min(mb, lo + per);
        if (lo < hi) pool.emplace_back(work, lo, hi);
    }
    for (auto& th : pool) th.join();
    return 0;
}

uint16_t orc_f32_to_bf16(float f) { return f32_to_bf16_rne(f); }

// The BLAS form of Sec. 2.2: C <- alpha * A*B + beta * C ("the scalars do not affect placement and the C read shares
// the partitioning of the output write").  Cin is the logical [M x N] bf16 matrix read; the fp32 sequential-k sum of
// orc_gemm is scaled and added to beta * Cin in double, then rounded once to fp32 (ref32) and to bf16 (out_bf16).
int orc_gemm_axpby(int64_t M, int64_t N, int64_t K, const uint16_t* A, int a_trans, const uint16_t* B, int b_trans,
                   double alpha, double beta, const uint16_t* Cin, float* ref32, uint16_t* out_bf16, int threads) {
    if (!Cin) return -1;
    std::vector<float> H((size_t)(M * N));
    if (orc_gemm(M, N, K, A, a_trans, B, b_trans, 0, M, 0, N, H.data(), nullptr, nullptr, threads)) return -1;
    for (int64_t i = 0; i < M * N; ++i) {
        const float v = (float)(alpha * (double)H[(size_t)i] + beta * (double)bf16_to_f32(Cin[i]));
        if (ref32) ref32[i] = v;
        if (out_bf16) out_bf16[i] = f32_to_bf16_rne(v);
    }
    return 0;
}

// Gated FFN activation on the product of a fused gate/up operand (the operand of Fig. 3; Sec. 3.3: activations are
// produced directly by upstream kernels).  H = A*B is [M x N], N even, its columns cut into P strips of width
// Wp = N/P (P = 1: one strip); strip g holds gate columns in its first half and up columns in its second half.
//   out[m][g*Wp/2 + j] = silu(H[m][g*Wp + j]) * H[m][g*Wp + Wp/2 + j],  0 <= j < Wp/2,  silu(x) = x / (1 + exp(-x)).
// H is the fp32 sequential-k sum of orc_gemm; silu and the product are evaluated in double from that fp32 value and
// rounded once to fp32 (ref32) and to bf16 (out_bf16).  The standard definition of the activation is used; the paper
// does not define one.
int orc_gemm_swiglu(int64_t M, int64_t N, int64_t K, int64_t P, const uint16_t* A, int a_trans, const uint16_t* B, int b_trans,
                    float* ref32, uint16_t* out_bf16, int threads) {
    if (M <= 0 || N <= 0 || K <= 0 || P < 1 || N % P || (N / P) % 2) return -1;
    std::vector<float> H((size_t)(M * N));
    if (orc_gemm(M, N, K, A, a_trans, B, b_trans, 0, M, 0, N, H.data(), nullptr, nullptr, threads)) return -1;
    const int64_t Wp = N / P, half = Wp / 2, No = N / 2;
    for (int64_t m = 0; m < M; ++m)
        for (int64_t g = 0; g < P; ++g)
            for (int64_t j = 0; j < half; ++j) {
                const double x = (double)H[(size_t)(m * N + g * Wp + j)], u = (double)H[(size_t)(m * N + g * Wp + half + j)];
                const float v = (float)(x / (1.0 + std::exp(-x)) * u);
                if (ref32) ref32[m * No + g * half + j] = v;
                if (out_bf16) out_bf16[m * No + g * half + j] = f32_to_bf16_rne(v);
            }
    return 0;
}

// Number of output tiles and of pages per operand.
int orc_traffic_sizes(const orc_traffic_desc* d, int64_t* ntiles, int64_t* pages) {
    if (!traffic_desc_ok(*d)) return -1;
    std::vector<Tile> tiles;
    std::vector<int32_t> zeros;
    const int32_t* q = nullptr;
    if (d->assign == ORC_ASSIGN_EXPLICIT) {   // count only: any valid assignment will do
        int64_t n = (int64_t)tile_dim(d->M, d->BM, d->P, false).size() * (int64_t)tile_dim(d->N, d->BN, d->P, false).size();
        zeros.assign((size_t)n, 0); q = zeros.data();
    }
    if (enumerate_tiles(*d, q, tiles)) return -1;
    *ntiles = (int64_t)tiles.size();
    pages[0] = pages_of(d->A, d->page_bytes); pages[1] = pages_of(d->B, d->page_bytes); pages[2] = pages_of(d->C, d->page_bytes);
    return 0;
}

// Tile rectangles and chiplets, [ntiles][5] = m0, m1, n0, n1, q (for sampling and tests).
int orc_traffic_tiles(const orc_traffic_desc* d, const int32_t* explicit_q, int64_t* out) {
    if (!traffic_desc_ok(*d)) return -1;
    std::vector<Tile> tiles;
    if (enumerate_tiles(*d, explicit_q, tiles)) return -1;
    for (size_t i = 0; i < tiles.size(); ++i) {
        out[i * 5 + 0] = tiles[i].m0; out[i * 5 + 1] = tiles[i].m1; out[i * 5 + 2] = tiles[i].n0; out[i * 5 + 3] = tiles[i].n1; out[i * 5 + 4] = tiles[i].q;
    }
    return 0;
}

// Remote-traffic count (Sec. 4.1 metric without the L2 filter), element by element.
//   per_cta  [ntiles][3 operands A,B,C][local, remote] bytes
//   per_page [X][pages_X][P] bytes of the page demanded by each chiplet (any entry may be NULL)
//   owner    [X][pages_X] chiplet the policy maps the page to
//   totals   [3][2]
int orc_traffic_elem(const orc_traffic_desc* d, const int32_t* explicit_q, uint64_t* per_cta, uint64_t* const* per_page,
                     uint8_t* const* owner, uint64_t* totals) {
    return traffic_impl<false>(*d, explicit_q, per_cta, per_page, owner, totals);
}

// Remote traffic behind an IDEAL private L2 per chiplet (a step towards the metric of Sec. 4.1, which counts
// only the reads that miss the chiplet's L2): a chiplet fetches every byte it needs at most once, however many of
// its CTAs touch it; output writes are counted once each.  Brute force: one "touched" bitmap per chiplet and
// operand, then every touched element is charged to local or remote by the owner of its page.
//   totals [3 operands][local, remote] bytes, summed over chiplets.  Fixed placements only (RR, BLOCK).
int orc_traffic_ideal_l2(const orc_traffic_desc* d, const int32_t* explicit_q, uint64_t* totals) {
    if (!traffic_desc_ok(*d)) return -1;
    std::vector<Tile> tiles;
    if (enumerate_tiles(*d, explicit_q, tiles)) return -1;
    const orc_mat* ms[3] = {&d->A, &d->B, &d->C};
    for (int i = 0; i < 6; ++i) totals[i] = 0;
    for (int X = 0; X < 3; ++X) {
        if (d->place[X] == ORC_PLACE_BEST) return -1;
        const orc_mat& m = *ms[X];
        int64_t n = buffer_elems(m), bytes_total = n * m.elem_bytes;
        for (int q = 0; q < d->P; ++q) {
            std::vector<uint8_t> touched((size_t)n, 0);
            for (const Tile& t : tiles) {
                if (t.q != q) continue;
                int64_t r0, r1, c0, c1; tile_rect(*d, t, X, r0, r1, c0, c1);
                for (int64_t r = r0; r < r1; ++r) for (int64_t c = c0; c < c1; ++c) touched[(size_t)map_offset(m, r, c)] = 1;
            }
            for (int64_t off = 0; off < n; ++off) {
                if (!touched[(size_t)off]) continue;
                int64_t page = off * m.elem_bytes / d->page_bytes;
                int32_t o = fixed_owner(d->place[X], page, d->page_bytes, d->P, bytes_total);
                totals[X * 2 + (o == q ? 0 : 1)] += (uint64_t)m.elem_bytes;
            }
        }
    }
    return 0;
}

// The same count taken run by run (a stored row of a tile is one contiguous run per strip,
// cut at page boundaries).  Validated against orc_traffic_elem in the tests; used at sizes
// where the element walk would take minutes.
// Remote traffic behind a FINITE private L2 per chiplet (Sec. 4.1: one L2 per chiplet, 8 MB, 128-byte lines,
// 16 ways; the metric counts operand reads from a remote chiplet that miss the L2, plus output writes to one).  What the paper
// leaves open is fixed here as the simplest tile-level model:
//   * every chiplet has its own cache of capacity_bytes / (line_bytes * ways) sets, LRU replacement inside a set;
//     the lines of A and of B are numbered from the start of their own buffers (assumed line-aligned) and carry the
//     operand in their tag; set index: hash = 0: line mod sets (the textbook index: power-of-two row pitches pile up
//     in a few sets); hash = 1: (line + H(line div sets)) mod sets with H(b) = high 32 bits of b * 0x9E3779B97F4A7C15
//     (a skew per block of `sets` consecutive lines, standing in for the address hashing of a real L2);
//   * the CTAs of a chiplet (its tiles, as enumerate_tiles assigns them) are taken in row-major order of the tile
//     grid (traversal 0: n fastest) or column-major (traversal 1: m fastest) and run in waves of wave_ctas
//     consecutive CTAs; the CTAs of a wave advance through K in lockstep, k_slice elements at a time (0: all of K):
//     for every k range, each CTA of the wave in turn touches every line of the A rows-by-k-range rectangle of its
//     tile in address order, then every line of its B rectangle; wave_ctas = 1, k_slice = 0 is one CTA after the
//     other, each reading all of A, then all of B;
//   * a hit costs nothing, a miss fetches the whole line from the page's owner: line_bytes local or remote bytes;
//     page_bytes must be a multiple of line_bytes;
//   * C is written once, past the cache: the C row of the totals is the one of the uncached count.
// Placement policies: RR and BLOCK.
typedef struct { int64_t capacity_bytes; int32_t line_bytes; int32_t ways; int32_t traversal; int32_t hash;
                 int32_t wave_ctas; int32_t k_slice; } orc_l2_model;

static int64_t lru_set_index(int64_t line, int64_t sets, int hash) {
    if (!hash) return line % sets;
    const uint64_t block = (uint64_t)(line / sets);
    const uint64_t skew = (block * 0x9E3779B97F4A7C15ull) >> 32;
    return (int64_t)(((uint64_t)(line % sets) + skew % (uint64_t)sets) % (uint64_t)sets);
}

int orc_traffic_lru(const orc_traffic_desc* d, const orc_l2_model* l2, uint64_t* totals) {
    if (!traffic_desc_ok(*d) || !l2) return -1;
    if (l2->line_bytes <= 0 || l2->ways <= 0 || l2->capacity_bytes <= 0 || (l2->traversal != 0 && l2->traversal != 1)) return -1;
    if (l2->hash != 0 && l2->hash != 1) return -1;
    if (l2->wave_ctas < 1 || l2->k_slice < 0) return -1;
    if (l2->capacity_bytes % ((int64_t)l2->line_bytes * l2->ways) || d->page_bytes % l2->line_bytes) return -1;
    if (d->assign == ORC_ASSIGN_EXPLICIT) return -1;
    const int64_t L = l2->line_bytes, sets = l2->capacity_bytes / (L * l2->ways);
    std::vector<Tile> tiles;
    if (enumerate_tiles(*d, nullptr, tiles)) return -1;
    const orc_mat* ms[3] = {&d->A, &d->B, &d->C};
    for (int i = 0; i < 6; ++i) totals[i] = 0;
    for (int X = 0; X < 3; ++X) if (d->place[X] == ORC_PLACE_BEST) return -1;
    // C: written once, uncached
    {
        const orc_mat& m = d->C;
        const int64_t bytes_total = buffer_elems(m) * m.elem_bytes;
        for (const Tile& t : tiles)
            for (int64_t r = t.m0; r < t.m1; ++r)
                for (int64_t c = t.n0; c < t.n1; ++c) {
                    const int64_t page = map_offset(m, r, c) * m.elem_bytes / d->page_bytes;
                    totals[4 + (fixed_owner(d->place[2], page, d->page_bytes, d->P, bytes_total) == t.q ? 0 : 1)] += (uint64_t)m.elem_bytes;
                }
    }
    // the order in which a chiplet runs its tiles
    std::vector<size_t> order(tiles.size());
    for (size_t i = 0; i < tiles.size(); ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](size_t a, size_t b) {
        const Tile &x = tiles[a], &y = tiles[b];
        if (l2->traversal == 0) return x.m0 != y.m0 ? x.m0 < y.m0 : x.n0 < y.n0;
        return x.n0 != y.n0 ? x.n0 < y.n0 : x.m0 < y.m0;
    });
    const int64_t W = l2->wave_ctas, ks = l2->k_slice > 0 ? l2->k_slice : d->K;
    for (int q = 0; q < d->P; ++q) {
        // cache[set] = tags from most to least recently used; tag = line * 2 + operand
        std::vector<std::vector<int64_t>> cache((size_t)sets);
        std::vector<size_t> mine;                       // this chiplet's tiles in the order it runs them
        for (size_t oi : order) if (tiles[oi].q == q) mine.push_back(oi);
        // waves of W tiles run in lockstep: every tile of the wave reads its A slice and its B slice of the k range
        // [k0, k0 + ks) before any of them moves on to the next range
        for (size_t w0 = 0; w0 < mine.size(); w0 += (size_t)W)
            for (int64_t k0 = 0; k0 < d->K; k0 += ks)
                for (size_t j = w0; j < std::min(mine.size(), w0 + (size_t)W); ++j) {
                    const Tile& t = tiles[mine[j]];
                    const int64_t k1 = std::min(d->K, k0 + ks);
                    for (int X = 0; X < 2; ++X) {
                        const orc_mat& m = *ms[X];
                        const int64_t bytes_total = buffer_elems(m) * m.elem_bytes;
                        int64_t r0, r1, c0, c1; tile_rect(*d, t, X, r0, r1, c0, c1);
                        const bool k_is_rows = X == 0 ? d->a_trans != 0 : d->b_trans == 0;
                        if (k_is_rows) { r0 = k0; r1 = k1; } else { c0 = k0; c1 = k1; }
                        std::vector<int64_t> lines;
                        for (int64_t r = r0; r < r1; ++r)
                            for (int64_t c = c0; c < c1; ++c) {
                                const int64_t b = map_offset(m, r, c) * m.elem_bytes;
                                lines.push_back(b / L);
                                lines.push_back((b + m.elem_bytes - 1) / L);
                            }
                        std::sort(lines.begin(), lines.end());
                        lines.erase(std::unique(lines.begin(), lines.end()), lines.end());
                        for (int64_t line : lines) {
                            std::vector<int64_t>& set = cache[(size_t)lru_set_index(line, sets, l2->hash)];
                            const int64_t tag = line * 2 + X;
                            auto it = std::find(set.begin(), set.end(), tag);
                            if (it != set.end()) { set.erase(it); set.insert(set.begin(), tag); continue; }      // hit
                            set.insert(set.begin(), tag);
                            if ((int64_t)set.size() > l2->ways) set.pop_back();
                            const int64_t page = line * L / d->page_bytes;
                            totals[X * 2 + (fixed_owner(d->place[X], page, d->page_bytes, d->P, bytes_total) == q ? 0 : 1)] += (uint64_t)L;
                        }
                    }
                }
    }
    return 0;
}

int orc_traffic_runs(const orc_traffic_desc* d, const int32_t* explicit_q, uint64_t* per_cta, uint64_t* const* per_page,
                     uint8_t* const* owner, uint64_t* totals) {
    return traffic_impl<true>(*d, explicit_q, per_cta, per_page, owner, totals);
}

}  // extern "C"
