// ccl_gemm: bf16 GEMM (fp32 accumulate, bf16 RNE output) whose A / B / C live in row-major or
// Chiplet-Contiguous Layout (Sec. 2.2 execution model; Sec. 3.3: only the address map changes).
//
// Design (sm_100a):
//   * CCL is folded into rank-3 TMA tensor maps {strip-local contiguous extent, rows, strip}
//     -- the view (K, G, N/G) with strides (w, K*w, 1) of Sec. 3.3 -- so the address
//     translation costs nothing per access and a partial last tile of a strip is handled by
//     TMA zero fill.
//   * One persistent CTA per SM, warp-specialised: warp 0 = TMA producer, warp 1 = tcgen05.mma
//     issuer (one elected thread) and TMEM owner, warps 2-5 = epilogue (TMEM -> registers ->
//     bf16 -> global, addressing C through its own layout).
//   * 128 x BN x 64 tiles (BN in {128,192,256}), SWIZZLE_128B shared-memory tiles, a ring of
//     smem stages, two TMEM accumulators so the epilogue of tile i overlaps the main loop of
//     tile i+1.
//   * Chiplet-grouped raster (Sec. 3.1): the CTAs are cut into P groups and group g walks only
//     the output tiles of strip g, i.e. it streams one contiguous region of B and C.
//   * Every mbarrier wait is bounded; on expiry the kernel records a code in g_gemm_status,
//     all roles leave their loops, TMEM is released and the kernel returns.
#include <algorithm>
#include <cstring>

#include <cuda_bf16.h>

#include "ccl_common.h"
#include "ccl_tma.h"

namespace ccl {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kGemmThreads = 192;
constexpr int kTmemCols = 512;
constexpr uint32_t kSmemBudget = 200 * 1024;   // ring of operand stages

__device__ int g_gemm_status = 0;

struct OpMap {          // how stored coordinates (r, c) of an operand become tensor-map coordinates
    int32_t split;      // 0 none, 1 rows, 2 cols
    int32_t w, h;       // strip width (split 2) / strip height (split 1)
};

struct GemmParams {
    int32_t M, N, K;
    int32_t Wm, Wn;                 // widths of the strips the tile grid respects (M / N when unsplit)
    int32_t tps_m, tps_n;           // tiles per strip
    int32_t tiles_m, tiles_n;
    int32_t num_kb;
    int32_t groups, group_dim;      // chiplet-grouped raster: number of CTA groups, 0 = along N, 1 = along M
    int32_t panel;                  // m-tiles per raster panel
    OpMap a, b;
    int32_t a_mn, b_mn;             // 1 = MN-major operand tile in shared memory
    int32_t c_split;
    int64_t c_w, c_h, c_stride, c_cols;
    uint16_t* C;
    uint32_t idesc;
    int32_t stages;
    uint32_t stage_bytes, a_bytes;  // bytes per stage, bytes of the A part
};

// ---- tcgen05 wrappers ---------------------------------------------------------------------
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, SWIZZLE_128B, descriptor version 1 (sm_100).
//   K-major : rows of 128 B (64 bf16 along K); 8-row groups every `sbo` bytes.
//   MN-major: rows of 128 B (64 bf16 along M/N), one row per k; 8-k groups every `sbo` bytes,
//             the next 64-element chunk along M/N every `lbo` bytes.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ void to_coords(const OpMap& o, int r, int c, int& x, int& y, int& z) {
    if (o.split == 2) { z = c / o.w; x = c - z * o.w; y = r; }
    else if (o.split == 1) { z = r / o.h; y = r - z * o.h; x = c; }
    else { x = c; y = r; z = 0; }
}

struct TileCoord { int m0, m1, n0, n1; };

// Tiles of this CTA: CTAs are cut into `groups` contiguous ranges; group g walks the tiles of its
// strip range in panels of `panel` m-tiles (m fastest inside a panel, then n, then the next panel).
struct Scheduler {
    const GemmParams& p;
    int gm, gn, tm_off, tn_off;     // sub-grid of this CTA's group
    int idx, step, bn;
    int64_t total;
    __device__ Scheduler(const GemmParams& p_, int bn_) : p(p_), bn(bn_) {
        int G = gridDim.x, c = blockIdx.x, g = 0, lo = 0, hi = G;
        if (p.groups > 1) {
            for (g = 0; g < p.groups; ++g) {
                lo = (int)(((int64_t)g * G) / p.groups);
                hi = (int)(((int64_t)(g + 1) * G) / p.groups);
                if (c >= lo && c < hi) break;
            }
        }
        idx = c - lo; step = hi - lo;
        gm = p.tiles_m; gn = p.tiles_n; tm_off = 0; tn_off = 0;
        if (p.groups > 1) {
            if (p.group_dim == 0) { gn = p.tiles_n / p.groups; tn_off = g * gn; }
            else { gm = p.tiles_m / p.groups; tm_off = g * gm; }
        }
        total = (int64_t)gm * gn;
    }
    __device__ bool get(int64_t i, TileCoord& t) const {
        if (i >= total) return false;
        int64_t per_panel = (int64_t)p.panel * gn;
        int pn = (int)(i / per_panel);
        int rem = (int)(i - (int64_t)pn * per_panel);
        int ph = min(p.panel, gm - pn * p.panel);
        int ln = rem / ph, lm = pn * p.panel + (rem - ln * ph);
        int tm = tm_off + lm, tn = tn_off + ln;
        int sm = tm / p.tps_m, jm = tm - sm * p.tps_m;
        int sn = tn / p.tps_n, jn = tn - sn * p.tps_n;
        t.m0 = sm * p.Wm + jm * BM; t.m1 = min(t.m0 + BM, (sm + 1) * p.Wm);
        t.n0 = sn * p.Wn; t.n1 = (sn + 1) * p.Wn;     // strip bounds; the BN step is applied by the caller
        t.n0 += jn * bn; t.n1 = min(t.n0 + bn, t.n1);
        return true;
    }
};

template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 1)
ccl_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const GemmParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)p.stages * p.stage_bytes);
    uint64_t* full = bars;
    uint64_t* empty = bars + p.stages;
    uint64_t* tmem_full = bars + 2 * p.stages;
    uint64_t* tmem_empty = tmem_full + 2;
    uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(tmem_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_ptr + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        prefetch_tmap(&map_a);
        prefetch_tmap(&map_b);
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&tmem_full[a], 1); mbar_init(&tmem_empty[a], 4); }
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(tmem_ptr, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr;

    Scheduler sched(p, BN);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            TileCoord t;
            bool ok = true;
            // K runs along the tensor map's x for a K-contiguous operand and along y otherwise.  Unless
            // the operand is split along K itself (rare), only that coordinate changes with kb, so
            // the box coordinates are computed once per tile.
            const bool a_ksplit = p.a_mn ? p.a.split == 1 : p.a.split == 2;
            const bool b_ksplit = p.b_mn ? p.b.split == 1 : p.b.split == 2;
            constexpr int NA = BM / 64, NB = BN / 64;
            for (int64_t i = sched.idx; ok && sched.get(i, t); i += sched.step) {
                int ax[NA], ay[NA], az[NA], bx[NB], by[NB], bz[NB];
                if (!p.a_mn) to_coords(p.a, t.m0, 0, ax[0], ay[0], az[0]);
                else {
#pragma unroll
                    for (int c = 0; c < NA; ++c) to_coords(p.a, 0, t.m0 + 64 * c, ax[c], ay[c], az[c]);
                }
                if (!p.b_mn) to_coords(p.b, t.n0, 0, bx[0], by[0], bz[0]);
                else {
#pragma unroll
                    for (int c = 0; c < NB; ++c) to_coords(p.b, 0, t.n0 + 64 * c, bx[c], by[c], bz[c]);
                }
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!mbar_wait_bounded(&empty[stage], phase ^ 1)) { atomicExch(&g_gemm_status, 1); *abort_flag = 1; ok = false; break; }
                    unsigned char* sa = smem + (size_t)stage * p.stage_bytes;
                    unsigned char* sb = sa + p.a_bytes;
                    mbar_expect_tx(&full[stage], p.stage_bytes);
                    const int k0 = kb * BK;
                    if (!p.a_mn) {                      // A stored [M x K]: one box of 64 k x 128 m
                        if (a_ksplit) to_coords(p.a, t.m0, k0, ax[0], ay[0], az[0]);
                        tma_load_3d(sa, &map_a, &full[stage], a_ksplit ? ax[0] : k0, ay[0], az[0]);
                    } else {                            // A stored [K x M]: boxes of 64 m x 64 k
#pragma unroll
                        for (int c = 0; c < NA; ++c) {
                            if (a_ksplit) to_coords(p.a, k0, t.m0 + 64 * c, ax[c], ay[c], az[c]);
                            tma_load_3d(sa + c * (64 * BK * 2), &map_a, &full[stage], ax[c], a_ksplit ? ay[c] : k0, az[c]);
                        }
                    }
                    if (!p.b_mn) {                      // B stored [N x K]: one box of 64 k x BN n
                        if (b_ksplit) to_coords(p.b, t.n0, k0, bx[0], by[0], bz[0]);
                        tma_load_3d(sb, &map_b, &full[stage], b_ksplit ? bx[0] : k0, by[0], bz[0]);
                    } else {                            // B stored [K x N]: boxes of 64 n x 64 k
#pragma unroll
                        for (int c = 0; c < NB; ++c) {
                            if (b_ksplit) to_coords(p.b, k0, t.n0 + 64 * c, bx[c], by[c], bz[c]);
                            tma_load_3d(sb + c * (64 * BK * 2), &map_b, &full[stage], bx[c], b_ksplit ? by[c] : k0, bz[c]);
                        }
                    }
                    if (++stage == p.stages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            TileCoord t;
            bool ok = true;
            int it = 0;
            // descriptor constants per operand
            const uint32_t a_lbo = p.a_mn ? 64 * BK * 2 : 16, b_lbo = p.b_mn ? 64 * BK * 2 : 16;
            const uint32_t a_kstep = p.a_mn ? (16 * 128) >> 4 : (16 * 2) >> 4;     // descriptor units (16 B) per UMMA_K = 16
            const uint32_t b_kstep = p.b_mn ? (16 * 128) >> 4 : (16 * 2) >> 4;
            for (int64_t i = sched.idx; ok && sched.get(i, t); i += sched.step, ++it) {
                const int acc = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1;
                if (!mbar_wait_bounded(&tmem_empty[acc], acc_phase ^ 1)) { atomicExch(&g_gemm_status, 2); *abort_flag = 1; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)acc * 256u;
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!mbar_wait_bounded(&full[stage], phase)) { atomicExch(&g_gemm_status, 3); *abort_flag = 1; ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + (size_t)stage * p.stage_bytes);
                    const uint64_t adesc = smem_desc(sa, a_lbo, 1024);
                    const uint64_t bdesc = smem_desc(sa + p.a_bytes, b_lbo, 1024);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        umma_bf16(tmem_d, adesc + (uint64_t)(k * a_kstep), bdesc + (uint64_t)(k * b_kstep), p.idesc, (kb | k) != 0);
                    umma_commit(&empty[stage]);          // frees the stage once these MMAs have read it
                    if (++stage == p.stages) { stage = 0; phase ^= 1; }
                }
                if (ok) umma_commit(&tmem_full[acc]);    // accumulator complete
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int quad = warp & 3;                       // TMEM lane quadrant this warp may read
        TileCoord t;
        int it = 0;
        for (int64_t i = sched.idx; sched.get(i, t); i += sched.step, ++it) {
            const int acc = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1;
            bool ok = mbar_wait_bounded(&tmem_full[acc], acc_phase);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { if (lane == 0) { atomicExch(&g_gemm_status, 4); *abort_flag = 1; } break; }
            tc_fence_after();
            const int m = t.m0 + quad * 32 + lane;
            // offset of (m, n) in C is row_base + n for every n of this tile
            int64_t row_base;
            if (p.c_split == 2) { int64_t g = t.n0 / p.c_w; row_base = g * p.c_stride + (int64_t)m * p.c_w - g * p.c_w; }
            else if (p.c_split == 1) { int64_t g = t.m0 / p.c_h; row_base = g * p.c_stride + ((int64_t)m - g * p.c_h) * p.c_cols; }
            else row_base = (int64_t)m * p.c_cols;
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)acc * 256u;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                if (t.n0 + c * 32 >= t.n1) break;        // warp-uniform: nothing valid further right
                uint32_t r[32];
                tmem_ld32(taddr + (uint32_t)(c * 32), r);
                tmem_ld_wait();
                if (m < t.m1) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int n = t.n0 + c * 32 + j * 8;
                        if (n < t.n1) {                  // n1 - n0 is a multiple of 8
                            uint4 v;
                            __nv_bfloat162 h;
                            h = __floats2bfloat162_rn(__uint_as_float(r[j * 8 + 0]), __uint_as_float(r[j * 8 + 1])); v.x = *reinterpret_cast<uint32_t*>(&h);
                            h = __floats2bfloat162_rn(__uint_as_float(r[j * 8 + 2]), __uint_as_float(r[j * 8 + 3])); v.y = *reinterpret_cast<uint32_t*>(&h);
                            h = __floats2bfloat162_rn(__uint_as_float(r[j * 8 + 4]), __uint_as_float(r[j * 8 + 5])); v.z = *reinterpret_cast<uint32_t*>(&h);
                            h = __floats2bfloat162_rn(__uint_as_float(r[j * 8 + 6]), __uint_as_float(r[j * 8 + 7])); v.w = *reinterpret_cast<uint32_t*>(&h);
                            *reinterpret_cast<uint4*>(p.C + row_base + n) = v;
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tmem_empty[acc]);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
struct GemmPlan {
    GemmParams p;
    int bn;
    MatView va, vb, vc;
    uint32_t smem_bytes;
    unsigned grid;
};

static ccl_status check_operand(const MatView& v, const void* ptr, const char* name) {
    if (v.e != 2) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: only 2-byte (bf16) elements are supported", name);
    int64_t inner = v.split == 2 ? v.w : v.cols;
    if (inner % 8) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: contiguous extent %lld is not a multiple of 8 elements", name, (long long)inner);
    if (v.split && (v.stride * v.e) % 16) return fail(CCL_ERR_ALIGN, "ccl_gemm: %s: strip stride is not a multiple of 16 bytes", name);
    if (ptr && (reinterpret_cast<uintptr_t>(ptr) & 15)) return fail(CCL_ERR_ALIGN, "ccl_gemm: %s: base pointer is not 16-byte aligned", name);
    if (v.rows >= (INT64_C(1) << 31) || v.cols >= (INT64_C(1) << 31) || v.stride * v.e >= (INT64_C(1) << 40))
        return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: extent too large for a tensor map", name);
    return CCL_OK;
}

// strip width an operand imposes on GEMM dimension `dim_is_rows ? stored rows : stored cols`
static int64_t split_width(const MatView& v, bool along_rows) {
    if (along_rows) return v.split == 1 ? v.h : 0;
    return v.split == 2 ? v.w : 0;
}

static ccl_status merge_width(int64_t* cur, int64_t w, const char* dim) {
    if (!w) return CCL_OK;
    if (*cur && *cur != w) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: operands split %s into strips of different widths (%lld vs %lld)", dim, (long long)*cur, (long long)w);
    *cur = w;
    return CCL_OK;
}

static ccl_status make_plan(const ccl_gemm_desc* d, const void* A, const void* B, const void* C, int sms, GemmPlan* plan) {
    if (!d) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm: NULL descriptor");
    if (d->M <= 0 || d->N <= 0 || d->K <= 0) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm: M, N, K must be positive");
    if (d->M >= (INT64_C(1) << 31) || d->N >= (INT64_C(1) << 31) || d->K >= (INT64_C(1) << 31)) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: dimension too large");
    if (d->out_part < 0 || d->out_part > 2) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm: unknown out_part");
    if (d->P < 1 || d->P > 255) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm: P must be in [1,255]");
    ccl_status s;
    if ((s = make_view(&d->A, "ccl_gemm: A", &plan->va))) return s;
    if ((s = make_view(&d->B, "ccl_gemm: B", &plan->vb))) return s;
    if ((s = make_view(&d->C, "ccl_gemm: C", &plan->vc))) return s;
    const MatView &va = plan->va, &vb = plan->vb, &vc = plan->vc;
    const bool at = d->a_trans != 0, bt = d->b_trans != 0;
    int64_t ar = at ? d->K : d->M, ac = at ? d->M : d->K, br = bt ? d->N : d->K, bc = bt ? d->K : d->N;
    if (va.rows != ar || va.cols != ac || vb.rows != br || vb.cols != bc || vc.rows != d->M || vc.cols != d->N)
        return fail(CCL_ERR_SHAPE, "ccl_gemm: operand shapes do not match M, N, K and the transpose flags");
    if ((s = check_operand(va, A, "A"))) return s;
    if ((s = check_operand(vb, B, "B"))) return s;
    if ((s = check_operand(vc, C, "C"))) return s;

    // strips along M, N (tiles must not straddle them) and along K (a 64-wide k block must not)
    int64_t Wm = 0, Wn = 0;
    if ((s = merge_width(&Wm, split_width(va, !at), "M"))) return s;
    if ((s = merge_width(&Wm, split_width(vc, true), "M"))) return s;
    if ((s = merge_width(&Wn, split_width(vb, bt), "N"))) return s;
    if ((s = merge_width(&Wn, split_width(vc, false), "N"))) return s;
    int groups = 1, group_dim = 0;
    if (d->grouped_raster && d->P > 1 && d->out_part != CCL_PART_NONE) {
        if (d->out_part == CCL_PART_COLS) {
            if (d->N % d->P) return fail(CCL_ERR_SHAPE, "ccl_gemm: N not divisible by P");
            if ((s = merge_width(&Wn, d->N / d->P, "N"))) return s;
            groups = d->P; group_dim = 0;
        } else {
            if (d->M % d->P) return fail(CCL_ERR_SHAPE, "ccl_gemm: M not divisible by P");
            if ((s = merge_width(&Wm, d->M / d->P, "M"))) return s;
            groups = d->P; group_dim = 1;
        }
    }
    int64_t ka = split_width(va, at), kb = split_width(vb, !bt);
    if ((ka && ka % BK) || (kb && kb % BK)) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: an operand split along K needs strips that are multiples of %d", BK);
    if (!Wm) Wm = d->M;
    if (!Wn) Wn = d->N;

    // BN: least padded work per strip, ties to the wider tile
    int best_bn = 256;
    int64_t best_waste = -1;
    for (int bn : {256, 192, 128}) {
        int64_t waste = (Wn + bn - 1) / bn * bn - Wn;
        if (best_waste < 0 || waste < best_waste) { best_waste = waste; best_bn = bn; }
    }
    plan->bn = best_bn;

    GemmParams& p = plan->p;
    std::memset(&p, 0, sizeof(p));
    p.M = (int32_t)d->M; p.N = (int32_t)d->N; p.K = (int32_t)d->K;
    p.Wm = (int32_t)Wm; p.Wn = (int32_t)Wn;
    p.tps_m = (int32_t)((Wm + BM - 1) / BM); p.tps_n = (int32_t)((Wn + best_bn - 1) / best_bn);
    p.tiles_m = (int32_t)(d->M / Wm) * p.tps_m; p.tiles_n = (int32_t)(d->N / Wn) * p.tps_n;
    p.num_kb = (int32_t)((d->K + BK - 1) / BK);
    p.a.split = va.split; p.a.w = (int32_t)va.w; p.a.h = (int32_t)va.h;
    p.b.split = vb.split; p.b.w = (int32_t)vb.w; p.b.h = (int32_t)vb.h;
    p.a_mn = at ? 1 : 0; p.b_mn = bt ? 0 : 1;
    p.c_split = vc.split; p.c_w = vc.w; p.c_h = vc.h; p.c_stride = vc.stride; p.c_cols = vc.cols;
    p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.a_mn << 15) | ((uint32_t)p.b_mn << 16) |
              ((uint32_t)(best_bn >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
    p.a_bytes = BM * BK * 2; p.stage_bytes = p.a_bytes + (uint32_t)best_bn * BK * 2;
    p.stages = (int32_t)(kSmemBudget / p.stage_bytes);
    if (p.stages > 8) p.stages = 8;
    p.panel = 16;
    int64_t ntiles = (int64_t)p.tiles_m * p.tiles_n;
    plan->grid = (unsigned)std::min<int64_t>(ntiles, sms);
    // grouped raster needs at least one CTA per group and whole strips per group
    if (groups > 1 && (int)plan->grid >= groups && (group_dim == 0 ? p.tiles_n % groups == 0 : p.tiles_m % groups == 0)) {
        p.groups = groups; p.group_dim = group_dim;
    } else { p.groups = 1; p.group_dim = 0; }
    plan->smem_bytes = (uint32_t)p.stages * p.stage_bytes + 1024 + (2 * p.stages + 4) * 8 + 16;
    return CCL_OK;
}

// tensor map of an operand: {contiguous extent, rows (per strip), strips}
static ccl_status operand_tmap(CUtensorMap* m, const MatView& v, const void* base, uint32_t box_inner, uint32_t box_rows) {
    uint64_t dims[3], strides[2];
    if (v.split == 2) { dims[0] = v.w; dims[1] = v.rows; dims[2] = v.nstrips; strides[0] = v.w * 2; strides[1] = v.stride * 2; }
    else if (v.split == 1) { dims[0] = v.cols; dims[1] = v.h; dims[2] = v.nstrips; strides[0] = v.cols * 2; strides[1] = v.stride * 2; }
    else { dims[0] = v.cols; dims[1] = v.rows; dims[2] = 1; strides[0] = v.cols * 2; strides[1] = v.cols * 2 * v.rows; }
    uint32_t box[3] = {box_inner, box_rows, 1};
    return encode_tmap(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

template <int BN>
static ccl_status launch(const GemmPlan& plan, const CUtensorMap& ma, const CUtensorMap& mb, cudaStream_t st) {
    static int configured_for = 0;
    if (configured_for < (int)plan.smem_bytes) {
        CCL_CUDA_TRY(cudaFuncSetAttribute(ccl_gemm_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes));
        configured_for = (int)plan.smem_bytes;
    }
    ccl_gemm_kernel<BN><<<plan.grid, kGemmThreads, plan.smem_bytes, st>>>(ma, mb, plan.p);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    return CCL_OK;
}

ccl_status repack_status_take(int* code);   // ccl_repack.cu

}  // namespace ccl

using namespace ccl;

extern "C" ccl_status ccl_gemm_workspace(const ccl_gemm_desc* d, size_t* bytes) {
    GemmPlan plan;
    ccl_status s = make_plan(d, nullptr, nullptr, nullptr, 148, &plan);
    if (s) return s;
    if (!bytes) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm_workspace: NULL output");
    *bytes = 0;
    return CCL_OK;
}

extern "C" ccl_status ccl_gemm(const ccl_gemm_desc* d, const void* A_dev, const void* B_dev, void* C_dev, void* ws_dev,
                               size_t ws_bytes, void* cuda_stream) {
    (void)ws_dev; (void)ws_bytes;
    if (!A_dev || !B_dev || !C_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm: NULL operand");
    GemmPlan plan;
    ccl_status s = make_plan(d, A_dev, B_dev, C_dev, 148, &plan);     // validation first: no CUDA call on bad input
    if (s) return s;
    int dev, sms;
    CCL_CUDA_TRY(cudaGetDevice(&dev));
    CCL_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    if ((s = make_plan(d, A_dev, B_dev, C_dev, sms, &plan))) return s;
    plan.p.C = static_cast<uint16_t*>(C_dev);
    CUtensorMap ma, mb;
    if (!plan.p.a_mn) s = operand_tmap(&ma, plan.va, A_dev, BK, BM); else s = operand_tmap(&ma, plan.va, A_dev, 64, BK);
    if (s) return s;
    if (!plan.p.b_mn) s = operand_tmap(&mb, plan.vb, B_dev, BK, (uint32_t)plan.bn); else s = operand_tmap(&mb, plan.vb, B_dev, 64, BK);
    if (s) return s;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    if (plan.bn == 256) return launch<256>(plan, ma, mb, st);
    if (plan.bn == 192) return launch<192>(plan, ma, mb, st);
    return launch<128>(plan, ma, mb, st);
}

extern "C" ccl_status ccl_gemm_status(void* cuda_stream, int32_t* detail) {
    CCL_CUDA_TRY(cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(cuda_stream)));
    int v = 0, z = 0, rv = 0;
    CCL_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_gemm_status, sizeof(int)));
    if (v) CCL_CUDA_TRY(cudaMemcpyToSymbol(g_gemm_status, &z, sizeof(int)));
    ccl_status s = repack_status_take(&rv);
    if (s) return s;
    if (detail) *detail = v ? v : (rv ? 100 + rv : 0);
    if (v || rv) return fail(CCL_ERR_TIMEOUT, "a bounded device-side wait expired (code %d)", v ? v : 100 + rv);
    return CCL_OK;
}
