// ccl_repack: row-major <-> CCL permutation copy (Sec. 3.3).
//
// Both directions are one strided 3-D copy over (strip g, row r of the strip, bytes of the row):
//   split along columns (Eq. 3): row-major side  g*w*e + r*C*e,   CCL side  g*stride*e + r*w*e
//   split along rows           : row-major side  g*h*C*e + r*C*e, CCL side  g*stride*e + r*C*e
// The work is pure HBM streaming (read once + write once).  Two kernels:
//   * repack_tma_kernel  -- one thread per CTA drives a ring of TMA tile loads and TMA tile
//     stores through shared memory (rank-3 tensor maps on both sides), so ~190 KB per SM
//     is in flight with no per-byte instruction cost.  Needs 16-byte alignment everywhere.
//   * repack_vec_kernel  -- plain vectorised loads/stores for every other shape
//     (vector width = the largest power of two that divides all extents and addresses).
#include <algorithm>
#include <cstdlib>
#include <cstring>

#include "ccl_common.h"
#include "ccl_tma.h"

namespace ccl {

struct CopyPlan {
    int64_t nstrips, rows, row_bytes;         // rows per strip, bytes per strip row
    int64_t src_g, src_r, dst_g, dst_r;       // byte strides
    int64_t pad_off, pad_bytes, pad_g;        // dir 0: zero dst[g*pad_g + pad_off, +pad_bytes) for every strip
    // page-interleaved CCL side (il_chunk = 0: none): byte b of strip g's packed contents lives at
    // g*il_chunk + (b / il_chunk)*il_chunk*il_P + b % il_chunk
    int64_t il_chunk, il_P;
    int32_t il_shift, il_dst;                 // log2(il_chunk) or -1; 1 = the destination is the interleaved side
    int64_t batch, src_b, dst_b;              // matrices per launch and the byte strides between them
    int64_t g0;                               // index of the first strip this launch covers (the narrower last strip of a
                                              // width that P does not divide is copied by a launch of its own)
};

__device__ __forceinline__ int64_t interleaved_off(const CopyPlan& p, int64_t g, int64_t b) {
    const int64_t j = p.il_shift >= 0 ? (b >> p.il_shift) : (b / p.il_chunk);
    return g * p.il_chunk + j * p.il_chunk * p.il_P + (b - j * p.il_chunk);
}

__device__ int g_repack_status = 0;

// ------------------------------------------------------------------------------------------
// Vector path
// ------------------------------------------------------------------------------------------
template <typename V>
__device__ __forceinline__ V ld_stream(const V* p) { return __ldcs(p); }
template <typename V>
__device__ __forceinline__ void st_stream(V* p, V v) { __stcs(p, v); }
template <>
__device__ __forceinline__ unsigned char ld_stream(const unsigned char* p) { return *p; }
template <>
__device__ __forceinline__ void st_stream(unsigned char* p, unsigned char v) { *p = v; }
template <>
__device__ __forceinline__ unsigned short ld_stream(const unsigned short* p) { return *p; }
template <>
__device__ __forceinline__ void st_stream(unsigned short* p, unsigned short v) { *p = v; }

constexpr int kVecThreads = 256;
constexpr int kVecUnroll = 4;

template <typename V, typename IDX>
__global__ void __launch_bounds__(kVecThreads) repack_vec_kernel(const char* __restrict__ src, char* __restrict__ dst, CopyPlan p,
                                                                 IDX chunks_per_row, IDX chunks_per_strip) {
    const int64_t g = blockIdx.y + p.g0;
    const char* s = src + (int64_t)blockIdx.z * p.src_b + g * p.src_g;
    char* d = dst + (int64_t)blockIdx.z * p.dst_b + g * p.dst_g;
    const IDX step = (IDX)gridDim.x * kVecThreads * kVecUnroll;
    for (IDX base = (IDX)blockIdx.x * kVecThreads * kVecUnroll + threadIdx.x; base < chunks_per_strip; base += step) {
        V v[kVecUnroll];
        int64_t doff[kVecUnroll];
        bool live[kVecUnroll];
#pragma unroll
        for (int u = 0; u < kVecUnroll; ++u) {
            IDX j = base + (IDX)u * kVecThreads;
            live[u] = j < chunks_per_strip;
            if (live[u]) {
                IDX r = j / chunks_per_row;
                IDX x = j - r * chunks_per_row;
                int64_t so = (int64_t)r * p.src_r + (int64_t)x * (int64_t)sizeof(V);
                int64_t dn = (int64_t)r * p.dst_r + (int64_t)x * (int64_t)sizeof(V);
                if (p.il_chunk) {                 // the CCL side is addressed through the chunk interleave
                    const int64_t b = (int64_t)r * p.row_bytes + (int64_t)x * (int64_t)sizeof(V);
                    if (p.il_dst) dn = interleaved_off(p, g, b) - g * p.dst_g; else so = interleaved_off(p, g, b) - g * p.src_g;
                }
                v[u] = ld_stream(reinterpret_cast<const V*>(s + so));
                doff[u] = dn;
            }
        }
#pragma unroll
        for (int u = 0; u < kVecUnroll; ++u)
            if (live[u]) st_stream(reinterpret_cast<V*>(d + doff[u]), v[u]);
    }
}

template <typename V>
__global__ void zero_pad_kernel(char* dst, int64_t pad_g, int64_t pad_off, int64_t chunks, int64_t dst_b) {
    char* d = dst + (int64_t)blockIdx.z * dst_b + (int64_t)blockIdx.y * pad_g + pad_off;
    V z;
    memset(&z, 0, sizeof(V));
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < chunks; i += (int64_t)gridDim.x * blockDim.x)
        reinterpret_cast<V*>(d)[i] = z;
}

// ------------------------------------------------------------------------------------------
// TMA path: tile = box of (bx 8-byte units) x (by rows) of one strip
// ------------------------------------------------------------------------------------------

struct TmaTiling {
    uint32_t bx, by;              // box extents (8-byte units, rows)
    uint32_t tiles_x, tiles_y;    // per strip
    uint32_t stages, stage_bytes; // ring depth and bytes per ring slot
    uint64_t ntiles;              // over all strips of all matrices of the batch
    // page-interleaved CCL side: which side it is and how a tile's (x, row, strip) becomes coordinates of its map.
    // il_mode 1: a chunk holds il_kr whole strip rows, map {x, row in chunk, strip, chunk};
    // il_mode 2: a strip row is whole chunks of il_s8 8-byte units, map {x in chunk, chunk in row, row, strip}.
    // The matrix of a batch is the coordinate after those (after {x, row, strip} on a plain side).
    uint32_t il_mode, il_src, il_kr, il_s8, nstrips;
};

struct Coord5 { int c[5]; };
__device__ __forceinline__ Coord5 tile_coord(const TmaTiling& t, bool il_side, uint32_t x, uint32_t y, uint32_t g, uint32_t b) {
    Coord5 r;
    if (!il_side) { r.c[0] = (int)x; r.c[1] = (int)y; r.c[2] = (int)g; r.c[3] = (int)b; r.c[4] = 0; }
    else if (t.il_mode == 1) { r.c[0] = (int)x; r.c[1] = (int)(y % t.il_kr); r.c[2] = (int)g; r.c[3] = (int)(y / t.il_kr); r.c[4] = (int)b; }
    else { r.c[0] = (int)(x % t.il_s8); r.c[1] = (int)(x / t.il_s8); r.c[2] = (int)y; r.c[3] = (int)g; r.c[4] = (int)b; }
    return r;
}

// After a wait on ring slot `it % stages` has run out: the loads of iterations it+1 .. (those issued so far) may still
// be in flight into this CTA's shared memory, and a CTA must not exit under them.  Gives each of them a further,
// short, bounded wait.  Loads are issued `stages` ahead at the start and then one per iteration, one iteration late
// (see the loop of repack_tma_kernel); `left` = iterations from `it` to the end of this CTA's tiles.
constexpr uint64_t kDrainLimitNs = 50000000ull;   // 50 ms per outstanding load
__device__ __forceinline__ void ring_drain(uint64_t* full, uint64_t it, uint32_t stages, uint64_t left) {
    const uint64_t issued_end = it == 0 ? stages : it + stages - 1;      // first iteration whose load is not issued yet
    for (uint64_t j = it + 1; j < issued_end && j - it < left; ++j)
        (void)mbar_wait_bounded(&full[j % stages], (uint32_t)((j / stages) & 1), kDrainLimitNs);
}

// RANK 3: one matrix, no interleaved side (maps {x, row, strip}); RANK 4: a batch of those, or one matrix with an
// interleaved side; RANK 5: a batch with an interleaved side.
template <int RANK>
__global__ void __launch_bounds__(32) repack_tma_kernel(const __grid_constant__ CUtensorMap src_map,
                                                           const __grid_constant__ CUtensorMap dst_map, TmaTiling t) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // stage buffers first (128-byte aligned), barriers after them
    unsigned char* stage0 = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    uint64_t* full = reinterpret_cast<uint64_t*>(stage0 + (size_t)t.stages * t.stage_bytes);
    if (threadIdx.x != 0) return;

    prefetch_tmap(&src_map);
    prefetch_tmap(&dst_map);
    for (int s = 0; s < t.stages; ++s) mbar_init(&full[s], 1);
    fence_barrier_init();

    const uint32_t box_bytes = t.bx * t.by * 8u;
    const uint64_t per_strip = (uint64_t)t.tiles_x * t.tiles_y;
    struct Tile { uint32_t x, y, g, b; };
    auto decode = [&](uint64_t tile) {
        Tile r;
        uint64_t gi = tile / per_strip;                       // strip index over the whole batch
        uint32_t rem = (uint32_t)(tile - gi * per_strip);
        uint32_t ty = rem / t.tiles_x, tx = rem - ty * t.tiles_x;
        r.x = tx * t.bx; r.y = ty * t.by;
        if (RANK == 3) { r.g = (uint32_t)gi; r.b = 0; }
        else { r.b = (uint32_t)(gi / t.nstrips); r.g = (uint32_t)(gi - (uint64_t)r.b * t.nstrips); }
        return r;
    };
    auto issue_load = [&](uint64_t it) {
        uint64_t tile = (uint64_t)blockIdx.x + it * gridDim.x;
        if (tile >= t.ntiles) return;
        uint32_t slot = (uint32_t)(it % t.stages);
        const Tile ti = decode(tile);
        void* buf = stage0 + (size_t)slot * t.stage_bytes;
        mbar_expect_tx(&full[slot], box_bytes);
        if (RANK == 3) tma_load_3d(buf, &src_map, &full[slot], (int)ti.x, (int)ti.y, (int)ti.g);
        else {
            const Coord5 c = tile_coord(t, t.il_mode && t.il_src, ti.x, ti.y, ti.g, ti.b);
            if (RANK == 4) tma_load_4d(buf, &src_map, &full[slot], c.c[0], c.c[1], c.c[2], c.c[3]);
            else tma_load_5d(buf, &src_map, &full[slot], c.c[0], c.c[1], c.c[2], c.c[3], c.c[4]);
        }
    };

    for (uint64_t it = 0; it < t.stages; ++it) issue_load(it);
    for (uint64_t it = 0;; ++it) {
        uint64_t tile = (uint64_t)blockIdx.x + it * gridDim.x;
        if (tile >= t.ntiles) break;
        uint32_t slot = (uint32_t)(it % t.stages);
        uint32_t parity = (uint32_t)((it / t.stages) & 1);
        if (!mbar_wait_bounded(&full[slot], parity)) {
            atomicExch(&g_repack_status, 1);
            // the loads already issued into the other slots may still be writing this CTA's shared memory
            ring_drain(full, it, t.stages, (t.ntiles - tile + gridDim.x - 1) / gridDim.x);
            break;
        }
        const Tile ti = decode(tile);
        const void* buf = stage0 + (size_t)slot * t.stage_bytes;
        if (RANK == 3) tma_store_3d(&dst_map, buf, (int)ti.x, (int)ti.y, (int)ti.g);
        else {
            const Coord5 c = tile_coord(t, t.il_mode && !t.il_src, ti.x, ti.y, ti.g, ti.b);
            if (RANK == 4) tma_store_4d(&dst_map, buf, c.c[0], c.c[1], c.c[2], c.c[3]);
            else tma_store_5d_bulk(&dst_map, buf, c.c[0], c.c[1], c.c[2], c.c[3], c.c[4]);
        }
        tma_store_commit();
        // the store issued one iteration ago has now read its buffer: refill that slot
        if (it >= 1) {
            tma_store_wait_read<1>();
            issue_load(it - 1 + t.stages);
        }
    }
    tma_store_wait_all<0>();
}

// ------------------------------------------------------------------------------------------
// Transposing repack: the source is the row-major TRANSPOSE [cols x rows] of the described matrix (a weight kept as
// [N x K] that a GEMM wants as CCL [K x N]); element (r, c) of the output comes from src[c * rows + r].
// ------------------------------------------------------------------------------------------
constexpr int kTrTile = 64, kTrThreads = 256, kTrStages = 4;
#ifndef CCL_TR_MIN_CTAS
#define CCL_TR_MIN_CTAS 5
#endif
constexpr int kTrMinCtas = CCL_TR_MIN_CTAS;

// 2-byte elements, everything a multiple of 8 elements: 64 x 64 tiles through 8 KB of shared memory.  A tile is read
// as 16-byte pieces of source rows (8 consecutive r at one c) and written as 16-byte pieces of output rows (8
// consecutive c at one r).  Shared memory holds the tile as [c][r] with the 16-byte granule index XORed with c / 8,
// which makes both the 16-byte stores of the first phase and the 2-byte gathers of the second free of bank conflicts.
__global__ void __launch_bounds__(kTrThreads, kTrMinCtas) repack_transpose_vec_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, MatView v,
                                                                          uint32_t tiles_c, uint32_t ntiles, int il_shift) {
    __shared__ __align__(16) uint16_t tile[kTrStages][kTrTile * kTrTile];
    const uint32_t t = threadIdx.x, q = t & 7, o = t >> 3;                  // q: 16-byte piece of a 128-byte row, o: 0..31
    const uint32_t rows = (uint32_t)v.rows, cols = (uint32_t)v.cols, w = (uint32_t)v.w;
    // A CTA takes a contiguous run of tiles, c fastest: it fills 64 output rows from left to right (its 128-byte
    // pieces of a row follow each other in time and leave L2 as whole rows), while the CTAs next to it read the
    // neighbouring pieces of the same source rows.
    const uint32_t first = (uint32_t)((uint64_t)ntiles * blockIdx.x / gridDim.x), last = (uint32_t)((uint64_t)ntiles * (blockIdx.x + 1) / gridDim.x);
    // source tiles arrive by 16-byte asynchronous copies straight into their (swizzled) place: kTrStages - 1 tiles
    // of reads stay in flight per CTA without holding registers
    uint32_t ltr = first / tiles_c, ltc = first - ltr * tiles_c;            // the next tile to load
    auto load_next = [&](uint32_t stage) {                                  // source row c0 + c, elements r0 + 8q .. + 8
        const uint32_t r = ltr * kTrTile + 8 * q;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const uint32_t cl = o + 32 * k, c = ltc * kTrTile + cl;
            const bool in = c < cols && r < rows;                           // outside: zero-filled (source size 0)
            const uint16_t* g = in ? src + (size_t)c * rows + r : src;
            const uint32_t sm = smem_u32(&tile[stage][cl * kTrTile + ((q ^ ((cl >> 3) & 7)) << 3)]);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(sm), "l"(g), "r"(in ? 16 : 0) : "memory");
        }
        if (++ltc == tiles_c) { ltc = 0; ++ltr; }
    };
#pragma unroll
    for (uint32_t d = 0; d < kTrStages - 1; ++d) {
        if (first + d < last) load_next(d);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    uint32_t tr = first / tiles_c, tc = first - tr * tiles_c, stage = 0;
    for (uint32_t ti = first; ti < last; ++ti) {
        asm volatile("cp.async.wait_group %0;" ::"n"(kTrStages - 2) : "memory");
        __syncthreads();                                                    // tile ti has landed; tile ti - 1 has been read out
        if (ti + kTrStages - 1 < last) load_next(stage == 0 ? kTrStages - 1 : stage - 1);
        asm volatile("cp.async.commit_group;" ::: "memory");
        // This thread writes 16-byte pieces (columns c .. c + 8) of the output rows r and r + 1: one 32-bit word of
        // shared memory holds both rows' elements of a column.
        const uint32_t c = tc * kTrTile + 8 * q, rl = 2 * o, r = tr * kTrTile + rl;
        if (c < cols && r < rows) {
            const uint32_t* tw = reinterpret_cast<const uint32_t*>(tile[stage]);
            uint32_t wd[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) wd[j] = tw[((8 * q + j) * kTrTile + ((((rl >> 3) ^ q) & 7) << 3) + (rl & 7)) >> 1];
            uint4 lo, hi;
            lo.x = __byte_perm(wd[0], wd[1], 0x5410); hi.x = __byte_perm(wd[0], wd[1], 0x7632);
            lo.y = __byte_perm(wd[2], wd[3], 0x5410); hi.y = __byte_perm(wd[2], wd[3], 0x7632);
            lo.z = __byte_perm(wd[4], wd[5], 0x5410); hi.z = __byte_perm(wd[4], wd[5], 0x7632);
            lo.w = __byte_perm(wd[6], wd[7], 0x5410); hi.w = __byte_perm(wd[6], wd[7], 0x7632);
            // offset of (r, c): packed strips of columns are Eq. 3 with one 32-bit division; rows are w apart
            int64_t off0, off1;
            if (v.split == 2) {
                const uint32_t g = c / w, cp = c - g * w;
                off0 = (int64_t)r * w + cp; off1 = off0 + w;
                if (v.ichunk) {                                             // chunk j of strip g is chunk j * P + g of the buffer
                    const int64_t j0 = il_shift >= 0 ? off0 >> il_shift : off0 / v.ichunk, j1 = il_shift >= 0 ? off1 >> il_shift : off1 / v.ichunk;
                    off0 = (j0 * v.nstrips + g) * v.ichunk + (off0 - j0 * v.ichunk);
                    off1 = (j1 * v.nstrips + g) * v.ichunk + (off1 - j1 * v.ichunk);
                } else { off0 += g * v.stride; off1 += g * v.stride; }
            } else { off0 = map(v, r, c); off1 = r + 1 < rows ? map(v, r + 1, c) : 0; }
            __stcs(reinterpret_cast<uint4*>(dst + off0), lo);
            if (r + 1 < rows) __stcs(reinterpret_cast<uint4*>(dst + off1), hi);
        }
        if (++tc == tiles_c) { tc = 0; ++tr; }
        if (++stage == kTrStages) stage = 0;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// Any element size and shape: 32 x 32 tiles, one element per access.
template <typename T>
__global__ void __launch_bounds__(kTrThreads) repack_transpose_elem_kernel(const T* __restrict__ src, T* __restrict__ dst, MatView v,
                                                                           int64_t tiles_r, int64_t ntiles) {
    __shared__ T tile[32][33];
    const int x = threadIdx.x & 31, y = threadIdx.x >> 5;                   // 8 rows of 32 threads
    for (int64_t ti = blockIdx.x; ti < ntiles; ti += gridDim.x) {
        const int64_t tc = ti / tiles_r, tr = ti - tc * tiles_r;
        const int64_t r0 = tr * 32, c0 = tc * 32;
        __syncthreads();
        for (int k = y; k < 32; k += 8)
            if (c0 + k < v.cols && r0 + x < v.rows) tile[k][x] = src[(c0 + k) * v.rows + r0 + x];
        __syncthreads();
        for (int k = y; k < 32; k += 8)
            if (r0 + k < v.rows && c0 + x < v.cols) dst[map(v, r0 + k, c0 + x)] = tile[x][k];
    }
}

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
static int64_t pow2_divisor(int64_t x, int64_t cap) {   // largest power of two <= cap dividing x (x = 0 -> cap)
    int64_t v = cap;
    while (v > 1 && (x % v)) v >>= 1;
    return v;
}

static int g_sm_count = 0;
static ccl_status sm_count(int* n) {
    if (!g_sm_count) {
        int dev;
        CCL_CUDA_TRY(cudaGetDevice(&dev));
        CCL_CUDA_TRY(cudaDeviceGetAttribute(&g_sm_count, cudaDevAttrMultiProcessorCount, dev));
    }
    *n = g_sm_count;
    return CCL_OK;
}

template <typename V>
static ccl_status launch_vec(const char* src, char* dst, const CopyPlan& p, int sms, cudaStream_t st) {
    int64_t cpr = p.row_bytes / (int64_t)sizeof(V), cps = cpr * p.rows;
    int64_t blocks_needed = (cps + (int64_t)kVecThreads * kVecUnroll - 1) / ((int64_t)kVecThreads * kVecUnroll);
    int64_t target = ((int64_t)sms * 8 + p.nstrips * p.batch - 1) / (p.nstrips * p.batch);
    dim3 grid((unsigned)std::max<int64_t>(1, std::min(blocks_needed, target)), (unsigned)p.nstrips, (unsigned)p.batch);
    if (cps < (INT64_C(1) << 31))
        repack_vec_kernel<V, uint32_t><<<grid, kVecThreads, 0, st>>>(src, dst, p, (uint32_t)cpr, (uint32_t)cps);
    else
        repack_vec_kernel<V, uint64_t><<<grid, kVecThreads, 0, st>>>(src, dst, p, (uint64_t)cpr, (uint64_t)cps);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    return CCL_OK;
}

template <typename V>
static ccl_status launch_pad(char* dst, const CopyPlan& p, cudaStream_t st) {
    int64_t chunks = p.pad_bytes / (int64_t)sizeof(V);
    dim3 grid((unsigned)std::max<int64_t>(1, std::min<int64_t>((chunks + 255) / 256, 64)), (unsigned)p.nstrips, (unsigned)p.batch);
    zero_pad_kernel<V><<<grid, 256, 0, st>>>(dst, p.pad_g, p.pad_off, chunks, p.dst_b);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    return CCL_OK;
}

static ccl_status launch_tma(const char* src, char* dst, const CopyPlan& p, int sms, cudaStream_t st) {
    uint64_t dims[3] = {(uint64_t)(p.row_bytes / 8), (uint64_t)p.rows, (uint64_t)p.nstrips};
    TmaTiling t;
    t.stages = 4; t.stage_bytes = 49152;                  // 4 x 48 KB measured best (6 x 32 KB: -3 %, 12 x 16 KB: -10 %)
    int ctas_per_sm = 1, max_bx = 256;
    t.bx = (uint32_t)std::min<uint64_t>((uint64_t)max_bx, dims[0]);
    t.il_mode = t.il_src = 0; t.il_kr = t.il_s8 = 1; t.nstrips = (uint32_t)p.nstrips;
    if (p.il_chunk) {
        t.il_src = p.il_dst ? 0 : 1;
        if (p.il_chunk % p.row_bytes == 0) { t.il_mode = 1; t.il_kr = (uint32_t)(p.il_chunk / p.row_bytes); }
        else {                                           // whole chunks per strip row: a box stays inside one chunk
            t.il_mode = 2; t.il_s8 = (uint32_t)(p.il_chunk / 8);
            while (t.il_s8 % t.bx || (t.bx & 1)) --t.bx;          // even: a TMA copy starts on a 16-byte boundary
        }
    }
    t.by = (uint32_t)std::max<uint64_t>(1, std::min<uint64_t>(std::min<uint64_t>(256, dims[1]), t.stage_bytes / (t.bx * 8ull)));
    uint32_t by_in = t.by, by_out = 1;                     // il_mode 1: rows of a box inside a chunk x chunks of a box
    if (t.il_mode == 1) {
        if (t.by >= t.il_kr) { by_in = t.il_kr; by_out = std::min<uint32_t>(t.by / t.il_kr, 256); }
        else { while (t.il_kr % by_in) --by_in; }
        t.by = by_in * by_out;
    }
    t.tiles_x = (uint32_t)((dims[0] + t.bx - 1) / t.bx);
    t.tiles_y = (uint32_t)((dims[1] + t.by - 1) / t.by);
    t.ntiles = (uint64_t)t.tiles_x * t.tiles_y * (uint64_t)p.nstrips * (uint64_t)p.batch;
    // a strip stride is irrelevant (and may be 0) when there is one strip, like the matrix stride of a batch of one:
    // give the encoder valid values
    const uint64_t src_g = (uint64_t)(p.nstrips > 1 ? p.src_g : p.src_r * p.rows), dst_g = (uint64_t)(p.nstrips > 1 ? p.dst_g : p.dst_r * p.rows);
    const uint64_t src_b = (uint64_t)(p.batch > 1 ? p.src_b : 16), dst_b = (uint64_t)(p.batch > 1 ? p.dst_b : 16);
    const int rank = 3 + (t.il_mode ? 1 : 0) + (p.batch > 1 ? 1 : 0);
    // every map is built with 5 dimensions and encoded with the first `rank` of them (the rest have extent 1)
    struct MapSpec { uint64_t dims[5], str[4]; uint32_t box[5]; };
    auto plain_side = [&](uint64_t row_stride, uint64_t g_stride, uint64_t b_stride) {
        MapSpec m = {{dims[0], dims[1], dims[2], (uint64_t)p.batch, 1}, {row_stride, g_stride, b_stride, 16}, {t.bx, t.by, 1, 1, 1}};
        return m;
    };
    auto il_side = [&](uint64_t b_stride) {
        const uint64_t S = (uint64_t)p.il_chunk, P = (uint64_t)p.il_P, chunks = ((uint64_t)p.rows * p.row_bytes + S - 1) / S;
        MapSpec m;
        if (t.il_mode == 1) {
            m = {{dims[0], t.il_kr, P, chunks, (uint64_t)p.batch}, {(uint64_t)p.row_bytes, S, S * P, b_stride}, {t.bx, by_in, 1, by_out, 1}};
        } else {
            const uint64_t cpr = (uint64_t)p.row_bytes / S;
            m = {{t.il_s8, cpr, dims[1], P, (uint64_t)p.batch}, {S * P, cpr * S * P, S, b_stride}, {t.bx, 1, t.by, 1, 1}};
        }
        return m;
    };
    const MapSpec ss = t.il_mode && t.il_src ? il_side(src_b) : plain_side((uint64_t)p.src_r, src_g, src_b);
    const MapSpec ds = t.il_mode && !t.il_src ? il_side(dst_b) : plain_side((uint64_t)p.dst_r, dst_g, dst_b);
    CUtensorMap sm, dm;
    ccl_status s = encode_tmap(&sm, CU_TENSOR_MAP_DATA_TYPE_UINT64, rank, src, ss.dims, ss.str, ss.box, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (s) return s;
    s = encode_tmap(&dm, CU_TENSOR_MAP_DATA_TYPE_UINT64, rank, dst, ds.dims, ds.str, ds.box, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (s) return s;
    size_t smem = (size_t)t.stages * t.stage_bytes + 128 + t.stages * sizeof(uint64_t);
    static size_t attr_set[3] = {0, 0, 0};
    const void* fn = rank == 3 ? (const void*)repack_tma_kernel<3> : rank == 4 ? (const void*)repack_tma_kernel<4> : (const void*)repack_tma_kernel<5>;
    if (attr_set[rank - 3] < smem) {
        CCL_CUDA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr_set[rank - 3] = smem;
    }
    unsigned grid = (unsigned)std::min<uint64_t>(t.ntiles, (uint64_t)sms * ctas_per_sm);
    if (rank == 3) repack_tma_kernel<3><<<grid, 32, smem, st>>>(sm, dm, t);
    else if (rank == 4) repack_tma_kernel<4><<<grid, 32, smem, st>>>(sm, dm, t);
    else repack_tma_kernel<5><<<grid, 32, smem, st>>>(sm, dm, t);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    return CCL_OK;
}

// Self-test of the expiry path of the ring above (ccl_selftest_wait_timeout, which = 1): the same ring of mbarriers,
// four slots of 512 bytes filled by plain bulk copies from src; the load of iteration 2 is left out on purpose, so the
// consumer's wait on it runs out after limit_ns, the status word gets its code, ring_drain() waits for the load of
// iteration 3 that is still outstanding, and the CTA returns.  Nothing waits on anything that cannot happen.
constexpr uint32_t kSelfSlots = 4, kSelfBytes = 512;
__global__ void __launch_bounds__(32) ring_selftest_kernel(const unsigned char* src, uint64_t limit_ns) {
    __shared__ __align__(128) unsigned char buf[kSelfSlots][kSelfBytes];
    __shared__ uint64_t full[kSelfSlots];
    if (threadIdx.x != 0) return;
    for (uint32_t s = 0; s < kSelfSlots; ++s) mbar_init(&full[s], 1);
    fence_barrier_init();
    for (uint32_t it = 0; it < kSelfSlots; ++it) {
        if (it == 2) continue;                                   // the load that never comes
        mbar_expect_tx(&full[it], kSelfBytes);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_u32(buf[it])), "l"(src + (size_t)it * kSelfBytes), "r"(kSelfBytes), "r"(smem_u32(&full[it])) : "memory");
    }
    for (uint64_t it = 0; it < kSelfSlots; ++it) {
        if (!mbar_wait_bounded(&full[it % kSelfSlots], 0u, limit_ns)) {
            atomicExch(&g_repack_status, 1);
            ring_drain(full, it, kSelfSlots, kSelfSlots - it);
            break;
        }
    }
}

ccl_status repack_selftest_launch(const void* src_dev, uint64_t limit_ns, cudaStream_t st) {
    if (!src_dev || (reinterpret_cast<uintptr_t>(src_dev) & 15))
        return fail(CCL_ERR_ALIGN, "ccl_selftest_wait_timeout: src_dev must be a 16-byte aligned device buffer of %u bytes", kSelfSlots * kSelfBytes);
    ring_selftest_kernel<<<1, 32, 0, st>>>(static_cast<const unsigned char*>(src_dev), limit_ns);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    return CCL_OK;
}

ccl_status repack_status_take(int* code) {
    int v = 0, z = 0;
    CCL_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_repack_status, sizeof(int)));
    if (v) CCL_CUDA_TRY(cudaMemcpyToSymbol(g_repack_status, &z, sizeof(int)));
    *code = v;
    return CCL_OK;
}

}  // namespace ccl

using namespace ccl;

// Where the padding of a CCL destination lies (p->nstrips, rows, row_bytes set): the tail of every aligned strip, or,
// page-interleaved, the tail of every strip's last chunk.
static void set_padding(const MatView& v, CopyPlan* p) {
    const int64_t e = v.e, Bs = p->rows * p->row_bytes;
    if (v.ichunk) {
        const int64_t S = v.ichunk * e;
        p->pad_g = S; p->pad_off = (v.ichunks - 1) * v.nstrips * S + (Bs - (v.ichunks - 1) * S); p->pad_bytes = v.ichunks * S - Bs;
    } else if (v.split) {
        p->pad_off = Bs; p->pad_bytes = v.stride * e - Bs; p->pad_g = v.stride * e;
    }
}

static ccl_status zero_padding(char* dst, const CopyPlan& p, cudaStream_t st) {
    if (p.pad_bytes <= 0) return CCL_OK;
    int64_t pv = pow2_divisor(p.pad_off | p.pad_bytes | p.pad_g | p.dst_b | (int64_t)(reinterpret_cast<uintptr_t>(dst) & 15), 16);
    if (pv == 16) return launch_pad<uint4>(dst, p, st);
    if (pv == 8) return launch_pad<uint2>(dst, p, st);
    if (pv == 4) return launch_pad<unsigned int>(dst, p, st);
    if (pv == 2) return launch_pad<unsigned short>(dst, p, st);
    return launch_pad<unsigned char>(dst, p, st);
}

static ccl_status repack_impl(const ccl_mat* m, int64_t batch, const void* src_dev, int64_t src_b, void* dst_dev, int64_t dst_b, int dir,
                              void* cuda_stream) {
    MatView v;
    ccl_status s = make_view(m, "ccl_repack", &v);
    if (s) return s;
    if (!src_dev || !dst_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_repack: NULL buffer");
    if (dir != 0 && dir != 1) return fail(CCL_ERR_INVALID_ARG, "ccl_repack: dir must be 0 or 1");
    if (src_dev == dst_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_repack: in-place repack is not supported");
    if ((reinterpret_cast<uintptr_t>(src_dev) % v.e) || (reinterpret_cast<uintptr_t>(dst_dev) % v.e))
        return fail(CCL_ERR_ALIGN, "ccl_repack: buffers must be aligned to elem_bytes");
    if (batch < 1 || batch > 65535) return fail(CCL_ERR_INVALID_ARG, "ccl_repack_batched: batch must be in [1, 65535]");
    if (batch > 1) {
        const int64_t plain = v.rows * v.cols * v.e, packed = buffer_elems(v) * v.e;
        if (src_b < 0 || dst_b < (dir == 0 ? packed : plain)) return fail(CCL_ERR_INVALID_ARG, "ccl_repack_batched: the outputs of a batch must not overlap (and strides must not be negative)");
        if (src_b % v.e || dst_b % v.e) return fail(CCL_ERR_ALIGN, "ccl_repack_batched: strides must be multiples of elem_bytes");
    } else src_b = dst_b = 0;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    int sms = 0;
    s = sm_count(&sms);
    if (s) return s;

    const int64_t e = v.e;
    CopyPlan p;
    std::memset(&p, 0, sizeof(p));
    p.batch = batch; p.src_b = src_b; p.dst_b = dst_b;
    int64_t rm_g, rm_r, cc_g, cc_r;          // row-major side and CCL side strides (bytes)
    if (v.split == 2) {
        p.nstrips = v.nstrips; p.rows = v.rows; p.row_bytes = v.w * e;
        rm_g = v.w * e; rm_r = v.cols * e; cc_g = v.stride * e; cc_r = v.w * e;
    } else if (v.split == 1) {
        p.nstrips = v.nstrips; p.rows = v.h; p.row_bytes = v.cols * e;
        rm_g = v.h * v.cols * e; rm_r = v.cols * e; cc_g = v.stride * e; cc_r = v.cols * e;
    } else {                                  // identity: a plain copy, treated as one strip
        p.nstrips = 1; p.rows = v.rows; p.row_bytes = v.cols * e;
        rm_g = 0; rm_r = v.cols * e; cc_g = 0; cc_r = v.cols * e;
    }
    if (p.nstrips > 65535) return fail(CCL_ERR_UNSUPPORTED, "ccl_repack: P > 65535");
    if (dir == 0) { p.src_g = rm_g; p.src_r = rm_r; p.dst_g = cc_g; p.dst_r = cc_r; }
    else          { p.src_g = cc_g; p.src_r = cc_r; p.dst_g = rm_g; p.dst_r = rm_r; }
    if (dir == 0) set_padding(v, &p);
    if (v.ichunk) {                           // page-interleaved CCL: chunk j of strip g is chunk j*P + g of the buffer
        const int64_t S = v.ichunk * e;
        p.il_chunk = S; p.il_P = v.nstrips; p.il_dst = dir == 0;
        p.il_shift = -1;
        if ((S & (S - 1)) == 0) { int sh = 0; while ((INT64_C(1) << sh) < S) ++sh; p.il_shift = sh; }
    }

    const char* src = static_cast<const char*>(src_dev);
    char* dst = static_cast<char*>(dst_dev);
    if (ragged(v)) {
        // The split dimension is not a multiple of P: the first P - 1 strips are one strided copy, the narrower (or
        // shorter) last strip another; padding (aligned strips, chunk tails) is cleared by zeroing the destination first.
        if (dir == 0 && (m->strip_align_bytes || v.ichunk))
            CCL_CUDA_TRY(cudaMemset2DAsync(dst, batch > 1 ? (size_t)dst_b : (size_t)(buffer_elems(v) * e), 0, (size_t)(buffer_elems(v) * e), (size_t)batch, st));
        for (int pass = 0; pass < 2; ++pass) {
            CopyPlan q = p;
            q.pad_bytes = 0;
            if (pass == 0) { q.nstrips = v.nstrips - 1; if (q.nstrips == 0) continue; }
            else {
                q.nstrips = 1; q.g0 = v.nstrips - 1;
                if (v.split == 2) {
                    q.row_bytes = v.wlast * e;
                    if (dir == 0) q.dst_r = v.wlast * e; else q.src_r = v.wlast * e;
                } else q.rows = v.hlast;
            }
            const int64_t addr = (int64_t)((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15);
            const int64_t vq = pow2_divisor(q.row_bytes | q.src_g | q.src_r | q.dst_g | q.dst_r | q.il_chunk | q.src_b | q.dst_b | addr, 16);
            if (vq == 16) s = launch_vec<uint4>(src, dst, q, sms, st);
            else if (vq == 8) s = launch_vec<uint2>(src, dst, q, sms, st);
            else if (vq == 4) s = launch_vec<unsigned int>(src, dst, q, sms, st);
            else if (vq == 2) s = launch_vec<unsigned short>(src, dst, q, sms, st);
            else s = launch_vec<unsigned char>(src, dst, q, sms, st);
            if (s) return s;
        }
        return CCL_OK;
    }
    int64_t addr_bits = (int64_t)((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15);
    int64_t vec = pow2_divisor(p.row_bytes | p.src_g | p.src_r | p.dst_g | p.dst_r | p.il_chunk | p.src_b | p.dst_b | addr_bits, 16);

    // path choice: TMA when everything is 16-byte aligned and the copy is big enough to be worth a ring
    const char* force = std::getenv("CCL_REPACK_PATH");
    // (page-interleaved side: a chunk must hold whole strip rows, or a strip row whole chunks)
    const bool il_ok = !p.il_chunk || p.il_chunk % p.row_bytes == 0 || p.row_bytes % p.il_chunk == 0;
    bool tma_ok = vec == 16 && il_ok && p.rows < (INT64_C(1) << 31) && p.row_bytes / 8 < (INT64_C(1) << 31) &&
                  std::max(std::max(std::max(p.src_g, p.src_r), std::max(p.dst_g, p.dst_r)), std::max(p.src_b, p.dst_b)) < (INT64_C(1) << 40);
    bool use_tma = tma_ok && p.batch * p.nstrips * p.rows * p.row_bytes >= (INT64_C(1) << 20);
    if (force && !std::strcmp(force, "vec")) use_tma = false;
    if (force && !std::strcmp(force, "tma") && tma_ok) use_tma = true;

    if (use_tma) s = launch_tma(src, dst, p, sms, st);
    else if (vec == 16) s = launch_vec<uint4>(src, dst, p, sms, st);
    else if (vec == 8) s = launch_vec<uint2>(src, dst, p, sms, st);
    else if (vec == 4) s = launch_vec<unsigned int>(src, dst, p, sms, st);
    else if (vec == 2) s = launch_vec<unsigned short>(src, dst, p, sms, st);
    else s = launch_vec<unsigned char>(src, dst, p, sms, st);
    if (s) return s;

    s = zero_padding(dst, p, st);
    if (s) return s;
    return CCL_OK;
}

extern "C" ccl_status ccl_repack(const ccl_mat* m, const void* src_dev, void* dst_dev, int dir, void* cuda_stream) {
    return repack_impl(m, 1, src_dev, 0, dst_dev, 0, dir, cuda_stream);
}

extern "C" ccl_status ccl_repack_batched(const ccl_mat* m, int32_t batch, const void* src_dev, int64_t src_stride_bytes, void* dst_dev,
                                         int64_t dst_stride_bytes, int dir, void* cuda_stream) {
    return repack_impl(m, batch, src_dev, src_stride_bytes, dst_dev, dst_stride_bytes, dir, cuda_stream);
}

extern "C" ccl_status ccl_repack_transpose(const ccl_mat* m, const void* src_dev, void* dst_dev, void* cuda_stream) {
    MatView v;
    ccl_status s = make_view(m, "ccl_repack_transpose", &v);
    if (s) return s;
    if (!src_dev || !dst_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_repack_transpose: NULL buffer");
    if (src_dev == dst_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_repack_transpose: in-place repack is not supported");
    if ((reinterpret_cast<uintptr_t>(src_dev) % v.e) || (reinterpret_cast<uintptr_t>(dst_dev) % v.e))
        return fail(CCL_ERR_ALIGN, "ccl_repack_transpose: buffers must be aligned to elem_bytes");
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    int sms = 0;
    s = sm_count(&sms);
    if (s) return s;
    CopyPlan p;
    std::memset(&p, 0, sizeof(p));
    p.batch = 1; p.nstrips = v.nstrips;
    if (v.split == 2) { p.rows = v.rows; p.row_bytes = v.w * v.e; }
    else if (v.split == 1) { p.rows = v.h; p.row_bytes = v.cols * v.e; }
    else { p.rows = v.rows; p.row_bytes = v.cols * v.e; }
    if (p.nstrips > 65535) return fail(CCL_ERR_UNSUPPORTED, "ccl_repack_transpose: P > 65535");
    set_padding(v, &p);
    char* dst = static_cast<char*>(dst_dev);
    const bool aligned16 = ((reinterpret_cast<uintptr_t>(src_dev) | reinterpret_cast<uintptr_t>(dst_dev)) & 15) == 0;
    if (ragged(v) && (m->strip_align_bytes || v.ichunk))      // strips of unequal size: the padding is cleared by zeroing the destination first
        CCL_CUDA_TRY(cudaMemsetAsync(dst, 0, (size_t)(buffer_elems(v) * v.e), st));
    const bool vec = !ragged(v) && v.e == 2 && aligned16 && v.rows % 8 == 0 && v.cols % 8 == 0 && v.w % 8 == 0 && v.stride % 8 == 0 && v.ichunk % 8 == 0 &&
                     v.rows < (INT64_C(1) << 31) && v.cols < (INT64_C(1) << 31) && ((v.rows + 63) / 64) * ((v.cols + 63) / 64) < (INT64_C(1) << 31);
    const int64_t T = vec ? kTrTile : 32;
    const int64_t tiles_r = (v.rows + T - 1) / T, tiles_c = (v.cols + T - 1) / T, ntiles = tiles_r * tiles_c;
    // a CTA takes a short run of tiles, all of whose reads it issues at once (the ring holds kTrStages - 1).  Measured
    // on the Llama weights: runs of 1: 4.1-4.5 TB/s, 2: 5.6-6.0, 3: 5.9-6.2, 4: 5.9-6.15, 6: 5.9, 24: 5.6
    int64_t run = kTrStages - 1;
    int il_shift = -1;
    if (v.ichunk && (v.ichunk & (v.ichunk - 1)) == 0) { il_shift = 0; while ((INT64_C(1) << il_shift) < v.ichunk) ++il_shift; }
    (void)sms;
    const unsigned grid = (unsigned)std::min<int64_t>((ntiles + run - 1) / run, INT64_C(1) << 30);
    static bool carveout_set = false;
    if (vec && !carveout_set) {                               // room for as many 32 KB rings per SM as registers allow
        CCL_CUDA_TRY(cudaFuncSetAttribute(repack_transpose_vec_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
        carveout_set = true;
    }
    if (vec) repack_transpose_vec_kernel<<<grid, kTrThreads, 0, st>>>(static_cast<const uint16_t*>(src_dev), reinterpret_cast<uint16_t*>(dst), v, (uint32_t)tiles_c, (uint32_t)ntiles, il_shift);
    else if (v.e == 1) repack_transpose_elem_kernel<uint8_t><<<grid, kTrThreads, 0, st>>>(static_cast<const uint8_t*>(src_dev), reinterpret_cast<uint8_t*>(dst), v, tiles_r, ntiles);
    else if (v.e == 2) repack_transpose_elem_kernel<uint16_t><<<grid, kTrThreads, 0, st>>>(static_cast<const uint16_t*>(src_dev), reinterpret_cast<uint16_t*>(dst), v, tiles_r, ntiles);
    else if (v.e == 4) repack_transpose_elem_kernel<uint32_t><<<grid, kTrThreads, 0, st>>>(static_cast<const uint32_t*>(src_dev), reinterpret_cast<uint32_t*>(dst), v, tiles_r, ntiles);
    else return fail(CCL_ERR_UNSUPPORTED, "ccl_repack_transpose: elem_bytes must be 1, 2 or 4");
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    return ragged(v) ? CCL_OK : zero_padding(dst, p, st);
}
