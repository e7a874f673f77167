// ccl_traffic: local / remote HBM byte counter (Sec. 4.1 metric without the L2 filter).
//
// Execution model (Sec. 2.2, Sec. 4.1): one CTA per BM x BN output tile; it reads its rows of
// A over all K, its columns of B over all K and writes its C tile.  Each operand's bytes are
// located through the operand's layout (Eq. 2 or Eq. 3), the page that holds them is mapped
// to a chiplet by the placement policy, and the bytes are local if that chiplet is the CTA's.
//
// Kernels (all integer):
//   prep      zero the outputs that are accumulated into
//   walk      every contiguous run a CTA touches is cut at strip and page boundaries; per piece the
//             per-page demand is accumulated and/or the piece is classified local / remote.  A is
//             walked once per tile row and B once per tile column (all tiles of the row / column
//             touch the same bytes), C once per tile
//   owner     page -> chiplet for every operand whose owner table is asked for / needed
#include <algorithm>
#include <cstring>

#include "ccl_common.h"

namespace ccl {

struct TrafficParams {
    int64_t M, N, K;
    int32_t BM, BN;
    MatView v[3];
    int32_t a_trans, b_trans, P;
    int64_t S;
    int32_t s_shift;              // log2(S) when S is a power of two, else -1
    int32_t place[3];
    int32_t assign;
    int32_t m_strip_tiled, n_strip_tiled;
    int64_t tiles_m, tiles_n, tps_m, tps_n, wM, wN;
    int32_t pm, pn;               // blocks of the output partition along M and N (pm * pn = P, or 1 x 1 for an explicit table)
    int64_t ntiles;
    int64_t pages[3];
    int64_t bytes_total[3];
    const int32_t* q;
    uint64_t* per_cta;
    uint64_t* per_page[3];
    uint8_t* owner[3];
    uint64_t* totals;
    uint64_t* totals_l2;          // optional: totals behind an ideal private L2 per chiplet (each byte fetched once per chiplet)
};

struct ZeroSeg { uint64_t* p[4]; int64_t n[4]; };

__global__ void traffic_prep_kernel(ZeroSeg z) {
    for (int s = 0; s < 4; ++s)
        for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < z.n[s]; i += (int64_t)gridDim.x * blockDim.x) z.p[s][i] = 0;
}

struct TileInfo { int64_t m0, m1, n0, n1; int32_t q; };

__device__ __forceinline__ TileInfo decode_tile(const TrafficParams& p, int64_t t) {
    TileInfo ti;
    int64_t tm = t / p.tiles_n, tn = t - tm * p.tiles_n;
    if (p.m_strip_tiled) {                        // strips of wM rows (the last one may be shorter), each tiled on its own
        int64_t g = min(tm / p.tps_m, (int64_t)p.pm - 1), j = tm - g * p.tps_m;
        ti.m0 = g * p.wM + j * p.BM; ti.m1 = min(ti.m0 + p.BM, min(p.M, (g + 1) * p.wM));
    } else { ti.m0 = tm * p.BM; ti.m1 = min(p.M, ti.m0 + p.BM); }
    if (p.n_strip_tiled) {
        int64_t g = min(tn / p.tps_n, (int64_t)p.pn - 1), j = tn - g * p.tps_n;
        ti.n0 = g * p.wN + j * p.BN; ti.n1 = min(ti.n0 + p.BN, min(p.N, (g + 1) * p.wN));
    } else { ti.n0 = tn * p.BN; ti.n1 = min(p.N, ti.n0 + p.BN); }
    // the block of the output partition that holds the tile's first element (N strips: 1 x P, M strips: P x 1)
    if (p.assign != CCL_ASSIGN_EXPLICIT) ti.q = (int32_t)((ti.m0 / p.wM) * p.pn + ti.n0 / p.wN);
    else { int32_t q = p.q[t]; ti.q = q < 0 ? 0 : (q >= p.P ? p.P - 1 : q); }
    return ti;
}

// stored-coordinate rectangle of operand X touched by a tile
__device__ __forceinline__ void tile_rect(const TrafficParams& p, const TileInfo& t, int X, int64_t& r0, int64_t& r1, int64_t& c0, int64_t& c1) {
    if (X == 0) { if (!p.a_trans) { r0 = t.m0; r1 = t.m1; c0 = 0; c1 = p.K; } else { r0 = 0; r1 = p.K; c0 = t.m0; c1 = t.m1; } }
    else if (X == 1) { if (!p.b_trans) { r0 = 0; r1 = p.K; c0 = t.n0; c1 = t.n1; } else { r0 = t.n0; r1 = t.n1; c0 = 0; c1 = p.K; } }
    else { r0 = t.m0; r1 = t.m1; c0 = t.n0; c1 = t.n1; }
}

// Walks the pieces (page, bytes) of one stored row segment [c0,c1) of row r.
template <class F>
__device__ __forceinline__ void walk_row(const TrafficParams& p, const MatView& v, int64_t r, int64_t c0, int64_t c1, F&& f) {
    int64_t c = c0;
    while (c < c1) {
        int64_t cend, off;
        if (v.split == 2) {
            int64_t g = c / v.w;
            cend = min(c1, (g + 1) * v.w);
            const int64_t wg = strip_w_of(v, g);   // the last strip of a ragged width has its own row pitch
            if (v.ichunk) {                        // page-interleaved CCL: contiguity also ends at every chunk
                const int64_t o = r * wg + (c - g * v.w);
                cend = min(cend, c + (o / v.ichunk + 1) * v.ichunk - o);
                off = interleave(v, g, o);
            } else off = g * v.stride + r * wg + (c - g * v.w);
        } else if (v.ichunk) {                     // split along rows, page-interleaved
            const int64_t g = r / v.h, o = (r - g * v.h) * v.cols + c;
            cend = min(c1, c + (o / v.ichunk + 1) * v.ichunk - o);
            off = interleave(v, g, o);
        } else {
            cend = c1;
            off = map(v, r, c);
        }
        int64_t b = off * v.e, bend = b + (cend - c) * v.e;
        int64_t page = p.s_shift >= 0 ? (b >> p.s_shift) : (b / p.S);
        while (b < bend) {
            int64_t pend = min(bend, (page + 1) * p.S);
            f(page, pend - b);
            b = pend;
            ++page;
        }
        c = cend;
    }
}

__device__ __forceinline__ int32_t fixed_owner(const TrafficParams& p, int X, int64_t page) {
    if (p.place[X] == CCL_PLACE_RR) return (int32_t)(page % p.P);
    int64_t o = (page * p.S * p.P) / p.bytes_total[X];
    return (int32_t)min((int64_t)(p.P - 1), o);
}

constexpr int kWalkThreads = 256;
constexpr int kWarpsPerBlock = kWalkThreads / 32;

// One pass over every byte the CTAs touch.  HIST accumulates the per-page demand, CLASSIFY the
// local / remote split.  The A rectangle of a tile depends only on its tile row and the B rectangle
// only on its tile column, so they are walked ONCE per tile row / column by a whole block, which
// records how many bytes each chiplet owns (and which chiplets the sharing tiles run on) and then
// hands every tile of the row / column its numbers; only C is walked per tile (one warp each).
//   blocks [0, tiles_m)                    : A of tile row j
//   blocks [tiles_m, tiles_m + tiles_n)    : B of tile column j
//   the rest                               : C, kWarpsPerBlock tiles per block
template <bool HIST, bool CLASSIFY>
__global__ void __launch_bounds__(kWalkThreads) traffic_walk_kernel(TrafficParams p) {
    __shared__ unsigned long long own[256];       // bytes of the rectangle whose page belongs to chiplet o
    __shared__ unsigned int cnt[256];             // tiles sharing the rectangle that run on chiplet q
    __shared__ unsigned long long blk[12];        // [0,6): totals, [6,12): totals behind the ideal L2
    const int tid = threadIdx.x, lane = tid & 31;
    const int64_t item = blockIdx.x;
    if (tid < 12) blk[tid] = 0;
    if (item < p.tiles_m + p.tiles_n) {
        const int X = item < p.tiles_m ? 0 : 1;
        const int64_t j = X == 0 ? item : item - p.tiles_m;
        const bool do_hist = HIST && p.per_page[X] != nullptr;
        if (!do_hist && !CLASSIFY) return;
        const int64_t nshare = X == 0 ? p.tiles_n : p.tiles_m;                  // tiles that touch this rectangle
        const int64_t t_first = X == 0 ? j * p.tiles_n : j, t_step = X == 0 ? 1 : p.tiles_n;
        for (int i = tid; i < p.P; i += kWalkThreads) { own[i] = 0; cnt[i] = 0; }
        __syncthreads();
        if (do_hist || p.totals_l2) {
            for (int64_t o = tid; o < nshare; o += kWalkThreads) atomicAdd(&cnt[decode_tile(p, t_first + o * t_step).q], 1u);
            __syncthreads();
        }
        const TileInfo ti = decode_tile(p, t_first);
        int64_t r0, r1, c0, c1;
        tile_rect(p, ti, X, r0, r1, c0, c1);
        const bool table = p.place[X] == CCL_PLACE_BEST;
        const uint8_t* own_tab = p.owner[X];
        unsigned long long* hist = reinterpret_cast<unsigned long long*>(p.per_page[X]);
        // bytes per owning chiplet: kept in registers while P <= 8 (the usual case; all threads of a block
        // tend to hit the same owner, which would serialise shared-memory atomics), else in shared memory
        const bool small_p = p.P <= 8;
        unsigned long long acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        for (int64_t r = r0 + tid; r < r1; r += kWalkThreads)
            walk_row(p, p.v[X], r, c0, c1, [&](int64_t page, int64_t len) {
                if (do_hist)
                    for (int q = 0; q < p.P; ++q) { const unsigned int n = cnt[q]; if (n) atomicAdd(&hist[page * p.P + q], (unsigned long long)len * n); }
                if (CLASSIFY) {
                    const int32_t o = table ? (int32_t)own_tab[page] : fixed_owner(p, X, page);
                    if (small_p) {
#pragma unroll
                        for (int q = 0; q < 8; ++q) acc[q] += (o == q) ? (unsigned long long)len : 0ull;
                    } else atomicAdd(&own[o], (unsigned long long)len);
                }
            });
        if (CLASSIFY && small_p) {
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                unsigned long long v = acc[q];
#pragma unroll
                for (int s2 = 16; s2 > 0; s2 >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s2);
                if (lane == 0 && v) atomicAdd(&own[q], v);
            }
        }
        if (CLASSIFY) {
            __syncthreads();
            unsigned long long total = 0, loc_sum = 0, rem_sum = 0;
            for (int o = 0; o < p.P; ++o) total += own[o];
            for (int64_t o = tid; o < nshare; o += kWalkThreads) {
                const int64_t t = t_first + o * t_step;
                const unsigned long long loc = own[decode_tile(p, t).q];
                if (p.per_cta) { p.per_cta[t * 6 + X * 2 + 0] = loc; p.per_cta[t * 6 + X * 2 + 1] = total - loc; }
                loc_sum += loc; rem_sum += total - loc;
            }
            if (p.totals_l2)                              // a chiplet fetches this rectangle once, however many of its tiles share it
                for (int q = tid; q < p.P; q += kWalkThreads)
                    if (cnt[q]) { atomicAdd(&blk[6 + X * 2 + 0], own[q]); atomicAdd(&blk[6 + X * 2 + 1], total - own[q]); }
            if (loc_sum) atomicAdd(&blk[X * 2 + 0], loc_sum);
            if (rem_sum) atomicAdd(&blk[X * 2 + 1], rem_sum);
        }
    } else {
        const int X = 2;
        const bool do_hist = HIST && p.per_page[X] != nullptr;
        if (!do_hist && !CLASSIFY) return;
        __syncthreads();                                  // blk[] zeroed
        const int64_t t = (item - p.tiles_m - p.tiles_n) * kWarpsPerBlock + (tid >> 5);
        if (t < p.ntiles) {
            const TileInfo ti = decode_tile(p, t);
            int64_t r0, r1, c0, c1;
            tile_rect(p, ti, X, r0, r1, c0, c1);
            const bool table = p.place[X] == CCL_PLACE_BEST;
            const uint8_t* own_tab = p.owner[X];
            unsigned long long* hist = reinterpret_cast<unsigned long long*>(p.per_page[X]);
            unsigned long long loc = 0, rem = 0;
            for (int64_t r = r0 + lane; r < r1; r += 32)
                walk_row(p, p.v[X], r, c0, c1, [&](int64_t page, int64_t len) {
                    if (do_hist) atomicAdd(&hist[page * p.P + ti.q], (unsigned long long)len);
                    if (CLASSIFY) {
                        const int32_t o = table ? (int32_t)own_tab[page] : fixed_owner(p, X, page);
                        if (o == ti.q) loc += (unsigned long long)len; else rem += (unsigned long long)len;
                    }
                });
            if (CLASSIFY) {
#pragma unroll
                for (int s = 16; s > 0; s >>= 1) {
                    loc += __shfl_xor_sync(0xffffffffu, loc, s);
                    rem += __shfl_xor_sync(0xffffffffu, rem, s);
                }
                if (lane == 0) {
                    if (p.per_cta) { p.per_cta[t * 6 + 4] = loc; p.per_cta[t * 6 + 5] = rem; }
                    atomicAdd(&blk[4], loc);
                    atomicAdd(&blk[5], rem);
                    atomicAdd(&blk[10], loc);                 // every output element is written once either way
                    atomicAdd(&blk[11], rem);
                }
            }
        }
    }
    if (CLASSIFY) {
        __syncthreads();
        if (tid < 6 && blk[tid] && p.totals) atomicAdd(reinterpret_cast<unsigned long long*>(p.totals) + tid, blk[tid]);
        if (tid >= 6 && tid < 12 && blk[tid] && p.totals_l2) atomicAdd(reinterpret_cast<unsigned long long*>(p.totals_l2) + (tid - 6), blk[tid]);
    }
}

__global__ void traffic_owner_kernel(TrafficParams p) {
    for (int X = 0; X < 3; ++X) {
        if (!p.owner[X]) continue;
        for (int64_t pg = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; pg < p.pages[X]; pg += (int64_t)gridDim.x * blockDim.x) {
            int32_t o;
            if (p.place[X] == CCL_PLACE_BEST) {
                const uint64_t* h = p.per_page[X] + pg * p.P;
                o = 0;
                uint64_t best = h[0];
                for (int q = 1; q < p.P; ++q) if (h[q] > best) { best = h[q]; o = q; }
            } else o = fixed_owner(p, X, pg);
            p.owner[X][pg] = (uint8_t)o;
        }
    }
}

// ---- finite private L2 per chiplet (tile-level LRU model) --------------------------------------------------
// Sec. 4.1 scores the operand reads from a remote chiplet that miss the L2, and the output writes to one, with an 8 MB,
// 16-way, 128-byte-line L2 per chiplet.  Model: the CTAs of a chiplet are taken in row-major (traversal 0) or column-major (traversal 1)
// order of the tile grid and run in waves of `wave` consecutive CTAs that step through K together, `ks` elements at
// a time; in each step every CTA of the wave in turn touches the lines of the k range of its A rectangle in address
// order, then those of its B rectangle (wave = 1, ks = K: one CTA after the other); lines are numbered from the start of each operand's buffer and the operand is part of the tag,
// LRU inside a set; a miss moves one whole line from the page's owner.
// Sets are independent, so one warp simulates one set of one chiplet over the whole run: it enumerates, tile by
// tile, only the lines that fall into its own set (32 blocks of lines per step) and lane 0 keeps the set's tags,
// most recently used first, in its own local array.  Set index: line mod sets, or (hash = 1) skewed per block of `sets` lines, which stands in for the
// address hashing of a real L2 (with the plain index, power-of-two row pitches pile up in a few sets).
struct LruParams {
    int64_t sets, ks;              // ks: elements of K a wave consumes per step (K: everything at once)
    int32_t line, ways, traversal, hash, wave;
    int32_t line_shift, sets_shift;   // log2 when a power of two, else -1
    uint64_t* out;                 // [2][2]: A local, A remote, B local, B remote
};

constexpr int kLruMaxWays = 32;
constexpr int kLruMaxWave = 256;
constexpr int kLruWarps = 4;       // warps (sets) per block

struct LruSet {
    uint64_t tag[kLruMaxWays];
    int n;
    // returns true on a miss
    __device__ __forceinline__ bool touch(uint64_t t, int ways) {
        int i = 0;
        while (i < n && tag[i] != t) ++i;
        const bool miss = i == n;
        if (miss) { if (n < ways) ++n; i = n - 1; }
        for (; i > 0; --i) tag[i] = tag[i - 1];
        tag[0] = t;
        return miss;
    }
};

__global__ void __launch_bounds__(32 * kLruWarps) traffic_lru_kernel(TrafficParams p, LruParams l) {
    // one WARP per (chiplet, set): the lanes scan 32 blocks of a piece at a time for the set's line, lane 0 owns the
    // set's state and applies the hits in address order
    const int lane = threadIdx.x & 31;
    const int64_t wid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (wid >= l.sets * p.P) return;                                        // whole warps leave together
    const int32_t q = (int32_t)(wid / l.sets);
    const int64_t s = wid - (int64_t)q * l.sets;
    const int64_t L = l.line;
    LruSet set;
    set.n = 0;
    uint64_t cnt[4] = {0, 0, 0, 0};
    auto hit_line = [&](int X, int64_t line) {                              // lane 0 only
        if (set.touch(((uint64_t)line << 1) | (uint64_t)X, l.ways)) {
            const int64_t b = line * L;
            const int64_t page = p.s_shift >= 0 ? (b >> p.s_shift) : (b / p.S);
            cnt[X * 2 + (fixed_owner(p, X, page) == q ? 0 : 1)] += (uint64_t)L;
        }
    };
    // The lines of rows [0, rows) of one contiguous piece that fall into this warp's set, in address order.
    // Every block of `sets` consecutive lines holds exactly one line of each set (the index is the line's position
    // in its block plus a skew that depends on the block only), so the piece is scanned block by block.
    auto piece = [&](int X, int64_t base, int64_t rows, int64_t pitch, int64_t len) {
        if (rows <= 0 || len <= 0) return;
        const int64_t last = base + (rows - 1) * pitch + len - 1;
        const int64_t l0 = l.line_shift >= 0 ? base >> l.line_shift : base / L, l1 = l.line_shift >= 0 ? last >> l.line_shift : last / L;
        for (int64_t blk0 = l.sets_shift >= 0 ? l0 >> l.sets_shift : l0 / l.sets; blk0 * l.sets <= l1; blk0 += 32) {
            const int64_t blk = blk0 + lane;
            const uint64_t h = l.hash ? ((uint64_t)blk * 0x9E3779B97F4A7C15ull) >> 32 : 0;
            int64_t pos;                                                     // position of the set's line in its block
            if (l.sets_shift >= 0) pos = (s - (int64_t)h) & (l.sets - 1);
            else { const int64_t skew = (int64_t)(h % (uint64_t)l.sets); pos = s - skew + (s < skew ? l.sets : 0); }
            const int64_t line = blk * l.sets + pos;
            bool in = line >= l0 && line <= l1;
            if (in) {
                // does the line [line*L, line*L + L) hold a byte of some row [base + r*pitch, + len) ?
                const int64_t b0 = line * L, b1 = b0 + L;
                int64_t r = b0 > base ? (b0 - base) / pitch : 0;             // the last row that starts at or before the line
                if (r >= rows) r = rows - 1;
                in = base + r * pitch < b1 && base + r * pitch + len > b0;
                if (!in && r + 1 < rows) in = base + (r + 1) * pitch < b1;   // or the next row starts inside it
            }
            unsigned hits = __ballot_sync(0xffffffffu, in);
            while (hits) {                                                   // ascending lanes = ascending addresses
                const int src = __ffs(hits) - 1;
                hits &= hits - 1;
                const int64_t ln = __shfl_sync(0xffffffffu, line, src);
                if (lane == 0) hit_line(X, ln);
            }
        }
    };
    // the k range [k0, k1) of tile t's rectangle of operand X
    auto slice = [&](const TileInfo& t, int X, int64_t k0, int64_t k1) {
        const MatView& v = p.v[X];
        int64_t r0, r1, c0, c1;
        tile_rect(p, t, X, r0, r1, c0, c1);
        const bool k_is_rows = X == 0 ? p.a_trans : !p.b_trans;
        if (k_is_rows) { r0 = k0; r1 = k1; } else { c0 = k0; c1 = k1; }
        if (v.split == 2) {                                           // strips of columns: one piece per strip touched
            for (int64_t g = c0 / v.w; g * v.w < c1; ++g) {
                const int64_t ca = max(c0, g * v.w), cb = min(c1, (g + 1) * v.w), wg = strip_w_of(v, g);
                piece(X, (g * v.stride + r0 * wg + (ca - g * v.w)) * v.e, r1 - r0, wg * v.e, (cb - ca) * v.e);
            }
        } else if (v.split == 1) {                                    // strips of rows
            for (int64_t g = r0 / v.h; g * v.h < r1; ++g) {
                const int64_t ra = max(r0, g * v.h), rb = min(r1, (g + 1) * v.h);
                piece(X, (g * v.stride + (ra - g * v.h) * v.cols + c0) * v.e, rb - ra, v.cols * v.e, (c1 - c0) * v.e);
            }
        } else piece(X, (r0 * v.cols + c0) * v.e, r1 - r0, v.cols * v.e, (c1 - c0) * v.e);
    };
    // The chiplet's tiles in traversal order, a wave at a time: the warp gathers the next `wave` of its tiles into
    // shared memory, then steps the whole wave through K.
    __shared__ int64_t wave_tiles[kLruWarps][kLruMaxWave][4];
    int64_t (*wt)[4] = wave_tiles[threadIdx.x >> 5];
    const int64_t inner = l.traversal == 0 ? p.tiles_n : p.tiles_m;
    int64_t o = 0, i = 0;
    for (int64_t pos = 0; pos < p.ntiles;) {
        int nw = 0;
        for (; pos < p.ntiles && nw < l.wave; ++pos) {
            const int64_t tm = l.traversal == 0 ? o : i, tn = l.traversal == 0 ? i : o;
            const TileInfo t = decode_tile(p, tm * p.tiles_n + tn);
            if (++i == inner) { i = 0; ++o; }
            if (t.q != q) continue;
            if (lane == 0) { wt[nw][0] = t.m0; wt[nw][1] = t.m1; wt[nw][2] = t.n0; wt[nw][3] = t.n1; }
            ++nw;
        }
        __syncwarp();
        for (int64_t k0 = 0; k0 < p.K; k0 += l.ks)
            for (int j = 0; j < nw; ++j) {
                TileInfo t;
                t.m0 = wt[j][0]; t.m1 = wt[j][1]; t.n0 = wt[j][2]; t.n1 = wt[j][3]; t.q = q;
                const int64_t k1 = min(p.K, k0 + l.ks);
                slice(t, 0, k0, k1);
                slice(t, 1, k0, k1);
            }
        __syncwarp();
    }
    if (lane == 0)
        for (int k = 0; k < 4; ++k)
            if (cnt[k]) atomicAdd(reinterpret_cast<unsigned long long*>(&l.out[k]), (unsigned long long)cnt[k]);
}

static ccl_status fill_params(const ccl_traffic_desc* d, TrafficParams* p) {
    if (!d) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic: NULL descriptor");
    std::memset(p, 0, sizeof(*p));
    if (d->M <= 0 || d->N <= 0 || d->K <= 0 || d->BM <= 0 || d->BN <= 0) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic: sizes must be positive");
    if (d->P < 1 || d->P > 255) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic: P must be in [1,255]");
    if (d->page_bytes <= 0) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic: page_bytes must be positive");
    if (d->assign < 0 || d->assign > 3) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic: unknown assign");
    const ccl_mat* ms[3] = {&d->A, &d->B, &d->C};
    const char* names[3] = {"ccl_traffic: A", "ccl_traffic: B", "ccl_traffic: C"};
    for (int X = 0; X < 3; ++X) {
        ccl_status s = make_view(ms[X], names[X], &p->v[X]);
        if (s) return s;
        if (d->place[X] < 0 || d->place[X] > 2) return fail(CCL_ERR_INVALID_ARG, "%s: unknown placement", names[X]);
        if (d->page_bytes % p->v[X].e) return fail(CCL_ERR_INVALID_ARG, "%s: page_bytes not a multiple of elem_bytes", names[X]);
        p->place[X] = d->place[X];
        p->bytes_total[X] = buffer_elems(p->v[X]) * p->v[X].e;
        p->pages[X] = (p->bytes_total[X] + d->page_bytes - 1) / d->page_bytes;
        if ((double)p->bytes_total[X] * d->P > 4.0e18) return fail(CCL_ERR_INVALID_ARG, "%s: buffer too large", names[X]);
    }
    int64_t ar = d->a_trans ? d->K : d->M, ac = d->a_trans ? d->M : d->K;
    int64_t br = d->b_trans ? d->N : d->K, bc = d->b_trans ? d->K : d->N;
    if (d->A.rows != ar || d->A.cols != ac || d->B.rows != br || d->B.cols != bc || d->C.rows != d->M || d->C.cols != d->N)
        return fail(CCL_ERR_SHAPE, "ccl_traffic: operand shapes do not match M, N, K and the transpose flags");
    // output partition: pm x pn blocks of ceil(M / pm) x ceil(N / pn) (the last ones hold what is left)
    int64_t pm = 1, pn = 1;
    if (d->assign == CCL_ASSIGN_N_STRIPS) pn = d->P;
    else if (d->assign == CCL_ASSIGN_M_STRIPS) pm = d->P;
    else if (d->assign == CCL_ASSIGN_2D) {
        if (d->part_m < 1 || d->P % d->part_m) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic: part_m (%d) must divide P (%d)", d->part_m, d->P);
        pm = d->part_m; pn = d->P / d->part_m;
    }
    p->M = d->M; p->N = d->N; p->K = d->K; p->BM = d->BM; p->BN = d->BN;
    p->wM = (d->M + pm - 1) / pm; p->wN = (d->N + pn - 1) / pn;
    if ((pn - 1) * p->wN >= d->N) return fail(CCL_ERR_SHAPE, "ccl_traffic: N (%lld) cannot be cut into %lld strips (one would be empty)", (long long)d->N, (long long)pn);
    if ((pm - 1) * p->wM >= d->M) return fail(CCL_ERR_SHAPE, "ccl_traffic: M (%lld) cannot be cut into %lld strips (one would be empty)", (long long)d->M, (long long)pm);
    p->pm = (int32_t)pm; p->pn = (int32_t)pn;
    p->a_trans = d->a_trans != 0; p->b_trans = d->b_trans != 0; p->P = d->P; p->S = d->page_bytes;
    p->s_shift = -1;
    if ((d->page_bytes & (d->page_bytes - 1)) == 0) { int sh = 0; while ((INT64_C(1) << sh) < d->page_bytes) ++sh; p->s_shift = sh; }
    p->assign = d->assign;
    p->m_strip_tiled = pm > 1 && d->strip_tiling;
    p->n_strip_tiled = pn > 1 && d->strip_tiling;
    p->tps_m = p->m_strip_tiled ? (p->wM + d->BM - 1) / d->BM : 0;
    p->tps_n = p->n_strip_tiled ? (p->wN + d->BN - 1) / d->BN : 0;
    const int64_t m_last = d->M - (pm - 1) * p->wM, n_last = d->N - (pn - 1) * p->wN;
    p->tiles_m = p->m_strip_tiled ? p->tps_m * (pm - 1) + (m_last + d->BM - 1) / d->BM : (d->M + d->BM - 1) / d->BM;
    p->tiles_n = p->n_strip_tiled ? p->tps_n * (pn - 1) + (n_last + d->BN - 1) / d->BN : (d->N + d->BN - 1) / d->BN;
    p->ntiles = p->tiles_m * p->tiles_n;
    return CCL_OK;
}

}  // namespace ccl

using namespace ccl;

extern "C" ccl_status ccl_traffic_sizes(const ccl_traffic_desc* d, int64_t* ntiles, int64_t pages[3]) {
    TrafficParams p;
    ccl_status s = fill_params(d, &p);
    if (s) return s;
    if (!ntiles || !pages) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic_sizes: NULL output");
    *ntiles = p.ntiles;
    for (int X = 0; X < 3; ++X) pages[X] = p.pages[X];
    return CCL_OK;
}

extern "C" ccl_status ccl_traffic(const ccl_traffic_desc* d, const int32_t* cta_chiplet_dev, uint64_t* per_cta_dev,
                                  uint64_t* const per_page_dev[3], uint8_t* const owner_dev[3], uint64_t* totals_dev,
                                  void* cuda_stream) {
    TrafficParams p;
    ccl_status s = fill_params(d, &p);
    if (s) return s;
    if (!per_cta_dev || !totals_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic: per_cta_dev and totals_dev are required");
    if (d->assign == CCL_ASSIGN_EXPLICIT && !cta_chiplet_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic: explicit assignment needs cta_chiplet_dev");
    bool need_hist = false, need_owner = false;
    for (int X = 0; X < 3; ++X) {
        p.per_page[X] = per_page_dev ? per_page_dev[X] : nullptr;
        p.owner[X] = owner_dev ? owner_dev[X] : nullptr;
        if (p.place[X] == CCL_PLACE_BEST && (!p.per_page[X] || !p.owner[X]))
            return fail(CCL_ERR_WORKSPACE, "ccl_traffic: CCL_PLACE_BEST needs per_page_dev[%d] and owner_dev[%d]", X, X);
        need_hist |= p.per_page[X] != nullptr;
        need_owner |= p.owner[X] != nullptr;
    }
    p.q = cta_chiplet_dev; p.per_cta = per_cta_dev; p.totals = totals_dev;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    int dev, sms;
    CCL_CUDA_TRY(cudaGetDevice(&dev));
    CCL_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));

    ZeroSeg z;
    std::memset(&z, 0, sizeof(z));
    z.p[0] = totals_dev; z.n[0] = 6;
    for (int X = 0; X < 3; ++X) if (p.per_page[X]) { z.p[1 + X] = p.per_page[X]; z.n[1 + X] = p.pages[X] * p.P; }
    traffic_prep_kernel<<<sms * 2, 256, 0, st>>>(z);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());

    bool any_best = false;
    for (int X = 0; X < 3; ++X) any_best |= p.place[X] == CCL_PLACE_BEST;
    const int64_t nblocks = p.tiles_m + p.tiles_n + (p.ntiles + kWarpsPerBlock - 1) / kWarpsPerBlock;
    if (nblocks >= (INT64_C(1) << 31)) return fail(CCL_ERR_UNSUPPORTED, "ccl_traffic: too many tiles");
    const unsigned grid = (unsigned)nblocks;
    if (any_best) {                       // demand first, then the owner table, then the classification that reads it
        traffic_walk_kernel<true, false><<<grid, kWalkThreads, 0, st>>>(p);
        count_launch();
        CCL_CUDA_TRY(cudaGetLastError());
        traffic_owner_kernel<<<sms * 2, 256, 0, st>>>(p);
        count_launch();
        CCL_CUDA_TRY(cudaGetLastError());
        traffic_walk_kernel<false, true><<<grid, kWalkThreads, 0, st>>>(p);
        count_launch();
        CCL_CUDA_TRY(cudaGetLastError());
    } else {
        if (need_hist) traffic_walk_kernel<true, true><<<grid, kWalkThreads, 0, st>>>(p);
        else traffic_walk_kernel<false, true><<<grid, kWalkThreads, 0, st>>>(p);
        count_launch();
        CCL_CUDA_TRY(cudaGetLastError());
        if (need_owner) {
            traffic_owner_kernel<<<sms * 2, 256, 0, st>>>(p);
            count_launch();
            CCL_CUDA_TRY(cudaGetLastError());
        }
    }
    return CCL_OK;
}

extern "C" ccl_status ccl_traffic_l2(const ccl_traffic_desc* d, const int32_t* cta_chiplet_dev, uint64_t* totals_l2_dev,
                                     void* cuda_stream) {
    TrafficParams p;
    ccl_status s = fill_params(d, &p);
    if (s) return s;
    if (!totals_l2_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic_l2: totals_l2_dev is required");
    if (d->assign == CCL_ASSIGN_EXPLICIT && !cta_chiplet_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic_l2: explicit assignment needs cta_chiplet_dev");
    for (int X = 0; X < 3; ++X)
        if (p.place[X] == CCL_PLACE_BEST) return fail(CCL_ERR_UNSUPPORTED, "ccl_traffic_l2: CCL_PLACE_BEST is not supported here (use a fixed placement)");
    p.q = cta_chiplet_dev; p.totals_l2 = totals_l2_dev;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    int dev, sms;
    CCL_CUDA_TRY(cudaGetDevice(&dev));
    CCL_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    ZeroSeg z;
    std::memset(&z, 0, sizeof(z));
    z.p[0] = totals_l2_dev; z.n[0] = 6;
    traffic_prep_kernel<<<1, 32, 0, st>>>(z);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    const int64_t nblocks = p.tiles_m + p.tiles_n + (p.ntiles + kWarpsPerBlock - 1) / kWarpsPerBlock;
    if (nblocks >= (INT64_C(1) << 31)) return fail(CCL_ERR_UNSUPPORTED, "ccl_traffic_l2: too many tiles");
    traffic_walk_kernel<false, true><<<(unsigned)nblocks, kWalkThreads, 0, st>>>(p);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    return CCL_OK;
}

extern "C" ccl_status ccl_traffic_lru(const ccl_traffic_desc* d, const ccl_l2_model* m, uint64_t* totals_dev, void* cuda_stream) {
    TrafficParams p;
    ccl_status s = fill_params(d, &p);
    if (s) return s;
    if (!m || !totals_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic_lru: NULL model or output");
    if (m->line_bytes <= 0 || m->ways <= 0 || m->capacity_bytes <= 0 || (m->traversal != 0 && m->traversal != 1))
        return fail(CCL_ERR_INVALID_ARG, "ccl_traffic_lru: line_bytes, ways, capacity_bytes must be positive and traversal 0 or 1");
    if (m->hash != 0 && m->hash != 1) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic_lru: hash must be 0 or 1");
    if (m->wave_ctas < 1 || m->k_slice < 0) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic_lru: wave_ctas must be at least 1 and k_slice non-negative");
    if (m->wave_ctas > kLruMaxWave) return fail(CCL_ERR_UNSUPPORTED, "ccl_traffic_lru: at most %d CTAs per wave", kLruMaxWave);
    if (m->ways > kLruMaxWays) return fail(CCL_ERR_UNSUPPORTED, "ccl_traffic_lru: at most %d ways", kLruMaxWays);
    if (m->capacity_bytes % ((int64_t)m->line_bytes * m->ways)) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic_lru: capacity is not a whole number of sets");
    if (d->page_bytes % m->line_bytes) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic_lru: page_bytes is not a multiple of line_bytes");
    if (d->assign == CCL_ASSIGN_EXPLICIT) return fail(CCL_ERR_UNSUPPORTED, "ccl_traffic_lru: explicit CTA assignment is not supported");
    for (int X = 0; X < 3; ++X) {
        if (p.place[X] == CCL_PLACE_BEST) return fail(CCL_ERR_UNSUPPORTED, "ccl_traffic_lru: CCL_PLACE_BEST is not supported here (use a fixed placement)");
        if (X < 2 && p.v[X].ichunk) return fail(CCL_ERR_UNSUPPORTED, "ccl_traffic_lru: page-interleaved operands are not supported");
    }
    LruParams l;
    std::memset(&l, 0, sizeof(l));
    l.line = m->line_bytes; l.ways = m->ways; l.traversal = m->traversal; l.hash = m->hash;
    l.line_shift = l.sets_shift = -1;
    l.wave = m->wave_ctas; l.ks = m->k_slice > 0 && m->k_slice < d->K ? m->k_slice : d->K;
    l.sets = m->capacity_bytes / ((int64_t)m->line_bytes * m->ways);
    for (int b = 0; b < 62; ++b) {
        if ((INT64_C(1) << b) == (int64_t)l.line) l.line_shift = b;
        if ((INT64_C(1) << b) == l.sets) l.sets_shift = b;
    }
    if (l.sets * d->P >= (INT64_C(1) << 31) * 128) return fail(CCL_ERR_UNSUPPORTED, "ccl_traffic_lru: too many sets");
    l.out = totals_dev;
    p.totals_l2 = totals_dev;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    ZeroSeg z;
    std::memset(&z, 0, sizeof(z));
    z.p[0] = totals_dev; z.n[0] = 6;
    traffic_prep_kernel<<<1, 32, 0, st>>>(z);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    // C is written once, past the cache: its row is the one of the walk behind an ideal L2 (= the uncached one)
    const int64_t nblocks = p.tiles_m + p.tiles_n + (p.ntiles + kWarpsPerBlock - 1) / kWarpsPerBlock;
    if (nblocks >= (INT64_C(1) << 31)) return fail(CCL_ERR_UNSUPPORTED, "ccl_traffic_lru: too many tiles");
    traffic_walk_kernel<false, true><<<(unsigned)nblocks, kWalkThreads, 0, st>>>(p);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    z.n[0] = 4;                                  // A and B come from the cache model
    traffic_prep_kernel<<<1, 32, 0, st>>>(z);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    const int64_t threads = l.sets * d->P * 32;          // a warp per (chiplet, set)
    traffic_lru_kernel<<<(unsigned)((threads + 32 * kLruWarps - 1) / (32 * kLruWarps)), 32 * kLruWarps, 0, st>>>(p, l);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    return CCL_OK;
}

