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
    const int64_t g = blockIdx.y;
    const char* s = src + g * p.src_g;
    char* d = dst + g * p.dst_g;
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
__global__ void zero_pad_kernel(char* dst, int64_t pad_g, int64_t pad_off, int64_t chunks) {
    char* d = dst + (int64_t)blockIdx.y * pad_g + pad_off;
    V z;
    memset(&z, 0, sizeof(V));
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < chunks; i += (int64_t)gridDim.x * blockDim.x)
        reinterpret_cast<V*>(d)[i] = z;
}

// ------------------------------------------------------------------------------------------
// TMA path: tile = box of (bx 8-byte units) x (by rows) of one strip
// ------------------------------------------------------------------------------------------
constexpr int kTmaMaxStages = 16;

struct TmaTiling {
    uint32_t bx, by;              // box extents (8-byte units, rows)
    uint32_t tiles_x, tiles_y;    // per strip
    uint32_t stages, stage_bytes; // ring depth and bytes per ring slot
    uint64_t ntiles;
    // page-interleaved CCL side (IL kernels): which side it is and how a tile's (x, row, strip) becomes coordinates
    // of its rank-4 map.  il_mode 1: a chunk holds il_kr whole strip rows, map {x, row in chunk, strip, chunk};
    // il_mode 2: a strip row is whole chunks of il_s8 8-byte units, map {x in chunk, chunk in row, row, strip}.
    uint32_t il_mode, il_src, il_kr, il_s8;
};

struct Coord4 { int c[4]; };
__device__ __forceinline__ Coord4 tile_coord(const TmaTiling& t, bool il_side, uint32_t x, uint32_t y, uint32_t g) {
    Coord4 r;
    if (!il_side) { r.c[0] = (int)x; r.c[1] = (int)y; r.c[2] = (int)g; r.c[3] = 0; }
    else if (t.il_mode == 1) { r.c[0] = (int)x; r.c[1] = (int)(y % t.il_kr); r.c[2] = (int)g; r.c[3] = (int)(y / t.il_kr); }
    else { r.c[0] = (int)(x % t.il_s8); r.c[1] = (int)(x / t.il_s8); r.c[2] = (int)y; r.c[3] = (int)g; }
    return r;
}

template <bool IL>
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
    auto issue_load = [&](uint64_t it) {
        uint64_t tile = (uint64_t)blockIdx.x + it * gridDim.x;
        if (tile >= t.ntiles) return;
        uint32_t slot = (uint32_t)(it % t.stages);
        uint32_t g = (uint32_t)(tile / per_strip);
        uint32_t rem = (uint32_t)(tile - (uint64_t)g * per_strip);
        uint32_t ty = rem / t.tiles_x, tx = rem - ty * t.tiles_x;
        mbar_expect_tx(&full[slot], box_bytes);
        if (IL) {
            const Coord4 c = tile_coord(t, t.il_src != 0, tx * t.bx, ty * t.by, g);
            tma_load_4d(stage0 + (size_t)slot * t.stage_bytes, &src_map, &full[slot], c.c[0], c.c[1], c.c[2], c.c[3]);
        } else
            tma_load_3d(stage0 + (size_t)slot * t.stage_bytes, &src_map, &full[slot], (int)(tx * t.bx), (int)(ty * t.by), (int)g);
    };

    for (uint64_t it = 0; it < t.stages; ++it) issue_load(it);
    for (uint64_t it = 0;; ++it) {
        uint64_t tile = (uint64_t)blockIdx.x + it * gridDim.x;
        if (tile >= t.ntiles) break;
        uint32_t slot = (uint32_t)(it % t.stages);
        uint32_t parity = (uint32_t)((it / t.stages) & 1);
        if (!mbar_wait_bounded(&full[slot], parity)) { atomicExch(&g_repack_status, 1); break; }
        uint32_t g = (uint32_t)(tile / per_strip);
        uint32_t rem = (uint32_t)(tile - (uint64_t)g * per_strip);
        uint32_t ty = rem / t.tiles_x, tx = rem - ty * t.tiles_x;
        if (IL) {
            const Coord4 c = tile_coord(t, t.il_src == 0, tx * t.bx, ty * t.by, g);
            tma_store_4d(&dst_map, stage0 + (size_t)slot * t.stage_bytes, c.c[0], c.c[1], c.c[2], c.c[3]);
        } else
            tma_store_3d(&dst_map, stage0 + (size_t)slot * t.stage_bytes, (int)(tx * t.bx), (int)(ty * t.by), (int)g);
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
    int64_t target = ((int64_t)sms * 8 + p.nstrips - 1) / p.nstrips;
    dim3 grid((unsigned)std::max<int64_t>(1, std::min(blocks_needed, target)), (unsigned)p.nstrips);
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
    dim3 grid((unsigned)std::max<int64_t>(1, std::min<int64_t>((chunks + 255) / 256, 64)), (unsigned)p.nstrips);
    zero_pad_kernel<V><<<grid, 256, 0, st>>>(dst, p.pad_g, p.pad_off, chunks);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    return CCL_OK;
}

static ccl_status launch_tma(const char* src, char* dst, const CopyPlan& p, int sms, cudaStream_t st) {
    uint64_t dims[3] = {(uint64_t)(p.row_bytes / 8), (uint64_t)p.rows, (uint64_t)p.nstrips};
    TmaTiling t;
    t.stages = 4; t.stage_bytes = 49152;                  // 4 x 48 KB measured best (6 x 32 KB: -3 %, 12 x 16 KB: -10 %)
    int ctas_per_sm = 1, max_bx = 256;
    if (const char* f = std::getenv("CCL_REPACK_TUNE")) {   // "stages,stage_kb,ctas_per_sm,max_bx"
        int a = 0, b = 0, c = 0, d2 = 0;
        if (sscanf(f, "%d,%d,%d,%d", &a, &b, &c, &d2) == 4 && a > 0 && a <= kTmaMaxStages && b > 0 && c > 0 && d2 > 0) { t.stages = a; t.stage_bytes = b * 1024; ctas_per_sm = c; max_bx = d2; }
    }
    t.bx = (uint32_t)std::min<uint64_t>((uint64_t)max_bx, dims[0]);
    t.il_mode = t.il_src = 0; t.il_kr = t.il_s8 = 1;
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
    t.ntiles = (uint64_t)t.tiles_x * t.tiles_y * (uint64_t)p.nstrips;
    // a strip stride is irrelevant (and may be 0) when there is one strip: give the encoder a valid value
    const uint64_t src_g = (uint64_t)(p.nstrips > 1 ? p.src_g : p.src_r * p.rows), dst_g = (uint64_t)(p.nstrips > 1 ? p.dst_g : p.dst_r * p.rows);
    CUtensorMap sm, dm;
    ccl_status s;
    if (!t.il_mode) {
        uint32_t box[3] = {t.bx, t.by, 1};
        uint64_t sstr[2] = {(uint64_t)p.src_r, src_g}, dstr[2] = {(uint64_t)p.dst_r, dst_g};
        s = encode_tmap(&sm, CU_TENSOR_MAP_DATA_TYPE_UINT64, 3, src, dims, sstr, box, CU_TENSOR_MAP_SWIZZLE_NONE);
        if (s) return s;
        s = encode_tmap(&dm, CU_TENSOR_MAP_DATA_TYPE_UINT64, 3, dst, dims, dstr, box, CU_TENSOR_MAP_SWIZZLE_NONE);
        if (s) return s;
    } else {
        // plain side: {x, row, strip, 1}; interleaved side: see TmaTiling.  Both boxes are by x bx dense in shared memory.
        const uint64_t S = (uint64_t)p.il_chunk, P = (uint64_t)p.il_P, chunks = ((uint64_t)p.rows * p.row_bytes + S - 1) / S;
        uint64_t pdims[4] = {dims[0], dims[1], dims[2], 1}, idims[4], istr[3];
        uint32_t pbox[4] = {t.bx, t.by, 1, 1}, ibox[4];
        if (t.il_mode == 1) {
            idims[0] = dims[0]; idims[1] = t.il_kr; idims[2] = P; idims[3] = chunks;
            istr[0] = (uint64_t)p.row_bytes; istr[1] = S; istr[2] = S * P;
            ibox[0] = t.bx; ibox[1] = by_in; ibox[2] = 1; ibox[3] = by_out;
        } else {
            const uint64_t m = (uint64_t)p.row_bytes / S;
            idims[0] = t.il_s8; idims[1] = m; idims[2] = dims[1]; idims[3] = P;
            istr[0] = S * P; istr[1] = m * S * P; istr[2] = S;
            ibox[0] = t.bx; ibox[1] = 1; ibox[2] = t.by; ibox[3] = 1;
        }
        const bool il_src = t.il_src != 0;
        uint64_t pstr[3] = {(uint64_t)(il_src ? p.dst_r : p.src_r), il_src ? dst_g : src_g, (il_src ? dst_g : src_g) * dims[2]};
        s = encode_tmap(&sm, CU_TENSOR_MAP_DATA_TYPE_UINT64, 4, src, il_src ? idims : pdims, il_src ? istr : pstr, il_src ? ibox : pbox, CU_TENSOR_MAP_SWIZZLE_NONE);
        if (s) return s;
        s = encode_tmap(&dm, CU_TENSOR_MAP_DATA_TYPE_UINT64, 4, dst, il_src ? pdims : idims, il_src ? pstr : istr, il_src ? pbox : ibox, CU_TENSOR_MAP_SWIZZLE_NONE);
        if (s) return s;
    }
    size_t smem = (size_t)t.stages * t.stage_bytes + 128 + t.stages * sizeof(uint64_t);
    static size_t attr_set[2] = {0, 0};
    const int which = t.il_mode ? 1 : 0;
    if (attr_set[which] < smem) {
        if (which) CCL_CUDA_TRY(cudaFuncSetAttribute(repack_tma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        else CCL_CUDA_TRY(cudaFuncSetAttribute(repack_tma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr_set[which] = smem;
    }
    unsigned grid = (unsigned)std::min<uint64_t>(t.ntiles, (uint64_t)sms * ctas_per_sm);
    if (which) repack_tma_kernel<true><<<grid, 32, smem, st>>>(sm, dm, t);
    else repack_tma_kernel<false><<<grid, 32, smem, st>>>(sm, dm, t);
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

extern "C" ccl_status ccl_repack(const ccl_mat* m, const void* src_dev, void* dst_dev, int dir, void* cuda_stream) {
    MatView v;
    ccl_status s = make_view(m, "ccl_repack", &v);
    if (s) return s;
    if (!src_dev || !dst_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_repack: NULL buffer");
    if (dir != 0 && dir != 1) return fail(CCL_ERR_INVALID_ARG, "ccl_repack: dir must be 0 or 1");
    if (src_dev == dst_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_repack: in-place repack is not supported");
    if ((reinterpret_cast<uintptr_t>(src_dev) % v.e) || (reinterpret_cast<uintptr_t>(dst_dev) % v.e))
        return fail(CCL_ERR_ALIGN, "ccl_repack: buffers must be aligned to elem_bytes");
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    int sms = 0;
    s = sm_count(&sms);
    if (s) return s;

    const int64_t e = v.e;
    CopyPlan p;
    std::memset(&p, 0, sizeof(p));
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
    if (dir == 0 && v.split && !v.ichunk) {
        p.pad_off = p.rows * p.row_bytes; p.pad_bytes = v.stride * e - p.pad_off; p.pad_g = cc_g;
    }
    if (v.ichunk) {                           // page-interleaved CCL: chunk j of strip g is chunk j*P + g of the buffer
        const int64_t S = v.ichunk * e, Bs = p.rows * p.row_bytes;
        p.il_chunk = S; p.il_P = v.nstrips; p.il_dst = dir == 0;
        p.il_shift = -1;
        if ((S & (S - 1)) == 0) { int sh = 0; while ((INT64_C(1) << sh) < S) ++sh; p.il_shift = sh; }
        if (dir == 0) {                       // the tail of every strip's last chunk is padding
            p.pad_g = S; p.pad_off = (v.ichunks - 1) * v.nstrips * S + (Bs - (v.ichunks - 1) * S); p.pad_bytes = v.ichunks * S - Bs;
        }
    }

    const char* src = static_cast<const char*>(src_dev);
    char* dst = static_cast<char*>(dst_dev);
    int64_t addr_bits = (int64_t)((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15);
    int64_t vec = pow2_divisor(p.row_bytes | p.src_g | p.src_r | p.dst_g | p.dst_r | p.il_chunk | addr_bits, 16);

    // path choice: TMA when everything is 16-byte aligned and the copy is big enough to be worth a ring
    const char* force = std::getenv("CCL_REPACK_PATH");
    // (page-interleaved side: a chunk must hold whole strip rows, or a strip row whole chunks)
    const bool il_ok = !p.il_chunk || p.il_chunk % p.row_bytes == 0 || p.row_bytes % p.il_chunk == 0;
    bool tma_ok = vec == 16 && il_ok && p.rows < (INT64_C(1) << 31) && p.row_bytes / 8 < (INT64_C(1) << 31) &&
                  std::max(std::max(p.src_g, p.src_r), std::max(p.dst_g, p.dst_r)) < (INT64_C(1) << 40);
    bool use_tma = tma_ok && p.nstrips * p.rows * p.row_bytes >= (INT64_C(1) << 20);
    if (force && !std::strcmp(force, "vec")) use_tma = false;
    if (force && !std::strcmp(force, "tma") && tma_ok) use_tma = true;

    if (use_tma) s = launch_tma(src, dst, p, sms, st);
    else if (vec == 16) s = launch_vec<uint4>(src, dst, p, sms, st);
    else if (vec == 8) s = launch_vec<uint2>(src, dst, p, sms, st);
    else if (vec == 4) s = launch_vec<unsigned int>(src, dst, p, sms, st);
    else if (vec == 2) s = launch_vec<unsigned short>(src, dst, p, sms, st);
    else s = launch_vec<unsigned char>(src, dst, p, sms, st);
    if (s) return s;

    if (p.pad_bytes > 0) {
        int64_t pv = pow2_divisor(p.pad_off | p.pad_bytes | p.pad_g | (int64_t)(reinterpret_cast<uintptr_t>(dst) & 15), 16);
        if (pv == 16) s = launch_pad<uint4>(dst, p, st);
        else if (pv == 8) s = launch_pad<uint2>(dst, p, st);
        else if (pv == 4) s = launch_pad<unsigned int>(dst, p, st);
        else if (pv == 2) s = launch_pad<unsigned short>(dst, p, st);
        else s = launch_pad<unsigned char>(dst, p, st);
        if (s) return s;
    }
    return CCL_OK;
}
