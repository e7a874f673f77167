// The GEMM kernel and what it shares with the host code that plans and launches it: tile constants, the parameter block,
// PTX wrappers (tcgen05, TMA, mbarrier, cluster), the tile walk, the kernel template and the split-K reduction.
// Included by ccl_gemm.cu only.
#ifndef CCL_GEMM_KERNEL_CUH_
#define CCL_GEMM_KERNEL_CUH_

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <atomic>
#include <mutex>

#include <cuda_bf16.h>

#include "ccl_common.h"
#include "ccl_tma.h"


namespace ccl {

constexpr int BM = 128;                         // rows of the output tile one CTA owns
constexpr int BK = 64;
#ifndef CCL_EPI_WARPS
#define CCL_EPI_WARPS 4
#endif
constexpr int kEpiWarps = CCL_EPI_WARPS;        // 4, or 8: two warps per TMEM lane quadrant taking alternate 64-column pieces
constexpr int kGemmThreads = 64 + 32 * kEpiWarps;
constexpr int kTmemCols = 512;
constexpr uint32_t kSmemBudget = 192 * 1024;    // ring of operand stages
constexpr int64_t kRaggedDense = 4096;         // problems of a ragged batch whose tile prefix is kept in shared memory
constexpr uint32_t kEpiBytes = 4 * 2 * 32 * 128; // epilogue staging: per warp two buffers of 32 rows x 128 B

__device__ int g_gemm_status = 0;
constexpr int kWaveSlots = 64;
__device__ unsigned int g_wave_ctr[kWaveSlots];

// Division of a non-negative int by a launch constant as a multiply-high and a shift (an integer division costs a few
// hundred cycles, and the tile walk of a short GEMM is nothing but divisions).  For d >= 2: l = ceil(log2 d),
// mul = ceil(2^(31+l) / d), n / d = umulhi(n, mul) >> (l - 1), exact for 0 <= n < 2^31; d = 1: mul = 0, shr = 0.
struct FastDiv {
    uint32_t d, mul, shr;
    __host__ __device__ int div(int n) const {
#ifdef __CUDA_ARCH__
        return mul ? (int)(__umulhi((uint32_t)n, mul) >> shr) : n;
#else
        return mul ? (int)(((uint64_t)(uint32_t)n * mul) >> 32 >> shr) : n;
#endif
    }
    __host__ __device__ void divmod(int n, int& q, int& r) const { q = div(n); r = n - q * (int)d; }
};
static FastDiv make_fastdiv(int64_t d) {
    FastDiv f;
    if (d < 1) d = 1;
    f.d = (uint32_t)d; f.mul = 0; f.shr = 0;
    if (d == 1) return f;
    int l = 0;
    while ((INT64_C(1) << l) < d) ++l;
    const unsigned __int128 one = 1;
    f.mul = (uint32_t)(((one << (31 + l)) + (unsigned __int128)d - 1) / (unsigned __int128)d);
    f.shr = (uint32_t)(l - 1);
    return f;
}

struct OpMap {          // how stored coordinates (r, c) of an operand become tensor-map coordinates
    int32_t split;      // 0 none, 1 rows, 2 cols
    FastDiv w, h;       // strip width (split 2) / strip height (split 1)
    // page-interleaved CCL (chunk of il_sc elements; chunk j of strip g stored as chunk j*P + g):
    //   il_mode 1: a chunk holds il_kr whole strip rows  -> map {x, row % kr, strip, row / kr}
    //   il_mode 2: a strip row spans whole chunks        -> map {x % sc, x / sc, row, strip}
    //   il_mode 0: strips stored one after the other     -> map {x, row, strip, 1}
    //   il_mode 3: neither (e.g. strip rows of 3.5 chunks): no affine box exists; a 64-element piece of a row at a
    //              64-aligned column is still contiguous, so the buffer is mapped as 128-byte lines {64, line} and a tile is
    //              fetched row by row (see line_of())
    int32_t il_mode;
    FastDiv il_kr, il_sc;
    int32_t batched;    // 1: each problem of a batch has its own buffer, 0: all problems share this operand
    int32_t rows, cols, roww, nstrips, lines;   // il_mode 3: stored shape, elements of a strip row, strips, 128-byte lines of the buffer
    int32_t rag;        // 1: the last strip is narrower / lower than the others (the split dimension is not a multiple of P):
                        // it has a tensor map of its own (the kernel's second set of maps), addressed with strip coordinate 0
};

struct GemmParams {
    int32_t M, N, K;
    int32_t Wm, Wn;                 // widths of the strips the tile grid respects (M / N when unsplit)
    int32_t tps_m, tps_n;           // tiles per strip (a tile is 128*CTAS x BN)
    int32_t tiles_m, tiles_n;
    int32_t num_kb;
    int32_t groups, group_dim;      // chiplet-grouped raster: number of CTA groups, 0 = along N, 1 = along M, 2 = blocks (2-D)
    int32_t groups_n;               // 2-D partition: blocks along N (group g owns block (g / groups_n, g % groups_n))
    FastDiv fd_groups_n;
    int32_t panel;                  // m-tiles per raster panel
    // raster constants the host derives from the grid it launches (see Scheduler)
    int32_t sch_units, sch_gm, sch_gn, sch_upg, sch_floaters, sch_rounds, sch_per_group, sch_pool_per_group;
    FastDiv fd_upg, fd_groups, fd_splits, fd_per_panel, fd_panel, fd_tps_m, fd_tps_n, fd_num_kb;
    // batch of independent problems of one shape (ccl_gemm_batched): the tile walk of a group runs through its
    // tiles of problem 0, then of problem 1, ...; problem e is coordinate e of every tensor map's last dimension
    int32_t batch;
    FastDiv fd_tiles_per_problem;   // tiles of one problem inside one group
    // gated activation (ccl_gemm_swiglu): N, Wn and the tile walk refer to the OUTPUT columns; the accumulators of a
    // tile hold the gate columns (sub-tile 0) and the up columns (sub-tile 1) of the same outputs, pair_dist B columns
    // apart inside a strip of 2 * pair_dist
    int32_t pair_dist;
    FastDiv fd_wn;
    // C <- alpha * A*B + beta * C (ccl_gemm_axpby); axpby = 0 when alpha = 1 and beta = 0 (C is then never read)
    int32_t axpby;
    float alpha, beta;
    int64_t c_batch_stride;         // elements between the C buffers of consecutive problems
    // ragged batch (ccl_gemm_grouped): problem e owns rows [m_offs[e], m_offs[e + 1]) of A and C; the tile grid of a
    // problem is laid out for Wm rows (the caller's bound) and tiles past a problem's last row are skipped
    // soft wave barrier (large problems): the producers of all CTAs meet here between full rounds of the tile walk, so
    // that the CTAs that share operand rows / columns stay close enough in time to find each other's lines in L2
    unsigned int* wave_ctr;
    int32_t wave_period, wave_wait_ns;
    const int32_t* m_offs;
    // ragged K (ccl_gemm_grouped_k): problem e contracts rows [k_offs[e], k_offs[e + 1]) of A [K x M] and B [K x N]
    const int32_t* k_offs;
    int32_t rag_dense;              // 1: the CTA builds a prefix of the problems' tile counts and walks only real tiles
    FastDiv fd_tiles_n;
    OpMap a, b;
    int32_t a_mn, b_mn;             // 1 = MN-major operand tile in shared memory
    OpMap c;                        // C addressed through its own map as well (TMA tile stores)
    int64_t c_row, c_stride, c_ichunk, c_nstrips;   // C: elements of a strip row, between strips, per chunk; strips
    int32_t c_cpr;                  // page-interleaved C whose strip rows span chunks: chunks per strip row
    uint16_t* C;
    int32_t c_wlast;                // elements of a row of C's last strip when that strip is narrower (else 0)
    uint32_t idesc;
    int32_t stages;
    uint32_t stage_bytes, a_bytes;  // bytes per stage per CTA, bytes of its A part
    uint32_t tx_bytes;              // bytes the copies of a stage deliver per CTA (stage_bytes unless the A box is cut short, see a_box_rows)
    int32_t splits, kb_per_split;   // split-K: each tile is computed by `splits` units over disjoint k-block ranges
    float* ws;                      // split-K partial sums, [splits][M][N] fp32 (row-major, logical coordinates)
    // balanced split: the k blocks of the first bal_tiles tiles of a group, laid end to end, are cut into equal shares, one
    // for each of the group's first bal_units units; bal_q / bal_r = quotient and remainder of that division
    int32_t bal, bal_q, bal_r, bal_units, bal_tiles;
    // cluster split: a cluster of `ks` CTAs computes ONE 128 x BN tile, CTA r of it the r-th kb_per_split k blocks; the
    // partial sums meet in distributed shared memory (see the epilogue)
    int32_t ks;
    // "partial sums written" flags, one per (CTA, epilogue warp), behind the partial sums in the workspace; zeroed by a
    // memset node in front of the launch (so a replayed CUDA graph clears them as well) and set to bal_mark by the kernel
    unsigned long long bal_mark;
    unsigned long long* bal_flags;
};

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

template <int CTAS>
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t ncols) {
    if (CTAS == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(ncols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    } else {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(ncols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
}
template <int CTAS>
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    if (CTAS == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
template <int CTAS>
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    if (CTAS == 1)
        asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                     ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
    else
        asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
                     ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// The four MMAs of one k block (UMMA_K = 16 each).  The MMA-issuing thread is the pacemaker of a short GEMM: its scalar
// instructions run one dependent step at a time, and ~300 cycles of address arithmetic, barrier polling and hand-back
// around ~300 cycles of MMA issue made every k block cost ~600 cycles whatever the tile width (measured), while a
// 256-wide block keeps the tensor pipe busy for 512.  So the descriptors are carried as 32-bit halves (only the low
// word, which holds the shared-memory address in 16-byte units, changes from step to step and from stage to stage),
// and, with PROBE, a look at the NEXT stage's barrier is started before the MMAs and read after them, so that its
// latency passes behind their issue.  Returns whether phase `probe_parity` of that barrier has completed (acquire).
// Called by a whole, converged warp with the same arguments in every lane (so that the compiler can keep them in
// uniform registers, which is where the MMA instruction takes its operands from); one elected lane issues the MMAs.
template <int CTAS, bool PROBE>
__device__ __forceinline__ uint32_t umma_bf16_x4(uint32_t tmem_d, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi, uint32_t a_kstep,
                                                 uint32_t b_kstep, uint32_t idesc, uint32_t accumulate, uint32_t probe_bar, uint32_t probe_parity) {
    uint32_t done = 0;
#define CCL_UMMA_X4(GROUP, PROBE_INSTR, PROBE_READ)                                                                     \
    asm volatile("{\n .reg .pred p, q, t, e;\n .reg .b32 x, y;\n .reg .b64 da, db;\n" PROBE_INSTR                         \
                 " elect.sync _|e, 0xffffffff;\n"                                                                        \
                 " setp.ne.b32 p, %9, 0;\n setp.eq.b32 t, 0, 0;\n"                                                       \
                 " mov.b64 da, {%2, %3};\n mov.b64 db, {%4, %5};\n"                                                      \
                 " @e tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], da, db, %8, p;\n"                                 \
                 " add.u32 x, %2, %6;\n add.u32 y, %4, %7;\n mov.b64 da, {x, %3};\n mov.b64 db, {y, %5};\n"             \
                 " @e tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], da, db, %8, t;\n"                                 \
                 " add.u32 x, x, %6;\n add.u32 y, y, %7;\n mov.b64 da, {x, %3};\n mov.b64 db, {y, %5};\n"               \
                 " @e tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], da, db, %8, t;\n"                                 \
                 " add.u32 x, x, %6;\n add.u32 y, y, %7;\n mov.b64 da, {x, %3};\n mov.b64 db, {y, %5};\n"               \
                 " @e tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], da, db, %8, t;\n" PROBE_READ "}"                  \
                 : "+r"(done)                                                                                            \
                 : "r"(tmem_d), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(a_kstep), "r"(b_kstep), "r"(idesc), "r"(accumulate),   \
                   "r"(probe_bar), "r"(probe_parity) : "memory")
    if (CTAS == 1 && PROBE) CCL_UMMA_X4("1", " mbarrier.test_wait.parity.shared::cta.b64 q, [%10], %11;\n", " selp.u32 %0, 1, 0, q;\n");
    else if (CTAS == 1) CCL_UMMA_X4("1", "", "");
    else if (PROBE) CCL_UMMA_X4("2", " mbarrier.test_wait.parity.shared::cta.b64 q, [%10], %11;\n", " selp.u32 %0, 1, 0, q;\n");
    else CCL_UMMA_X4("2", "", "");
#undef CCL_UMMA_X4
    return done;
}
// Arrive on an mbarrier once every MMA issued so far by this thread has completed.  With two CTAs
// the arrival is delivered to the barrier at the same offset in both CTAs of the pair.
template <int CTAS>
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    if (CTAS == 1)
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
    else
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                     ::"r"(smem_u32(bar)), "h"((unsigned short)3) : "memory");
}
// (called by a whole, converged warp: one elected lane issues the commit)
template <int CTAS>
__device__ __forceinline__ void umma_commit_addr(uint32_t bar_addr) {
    if (CTAS == 1)
        asm volatile("{\n .reg .pred e;\n elect.sync _|e, 0xffffffff;\n @e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}" ::"r"(bar_addr) : "memory");
    else
        asm volatile("{\n .reg .pred e;\n elect.sync _|e, 0xffffffff;\n @e tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n}"
                     ::"r"(bar_addr), "h"((unsigned short)3) : "memory");
}
// TMA tile load whose completion bytes are credited to `bar_addr` (a shared::cluster address; with two
// CTAs this is the leader's barrier, which the cta_group::2 form of the copy is allowed to signal).
template <int CTAS>
__device__ __forceinline__ void tma_load(void* smem_dst, const CUtensorMap* map, uint32_t bar_addr, int c0, int c1, int c2, int c3, int c4) {
    if (CTAS == 1)
        asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
                     ::"r"(smem_u32(smem_dst)), "l"(map), "r"(bar_addr), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
    else
        asm volatile("cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
                     ::"r"(smem_u32(smem_dst)), "l"(map), "r"(bar_addr), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
}
__device__ __forceinline__ void tma_store_5d(const CUtensorMap* map, const void* smem_src, int c0, int c1, int c2, int c3, int c4) {
    asm volatile("cp.async.bulk.tensor.5d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5, %6}], [%1];"
                 ::"l"(map), "r"(smem_u32(smem_src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
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
// 16-byte global store under a predicate, without a branch: the epilogue's TMEM loads and waits are warp-wide
// (.sync.aligned) and must never be reached by a warp that the compiler has split by a per-lane row test.
__device__ __forceinline__ void st_global_v4_if(void* ptr, uint4 v, bool pred) {
    asm volatile("{\n .reg .pred q;\n setp.ne.b32 q, %5, 0;\n @q st.global.v4.b32 [%0], {%1, %2, %3, %4};\n}"
                 ::"l"(ptr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"((uint32_t)pred) : "memory");
}
// 16-byte global load under a predicate (zeros when it is off), without a branch
__device__ __forceinline__ uint4 ld_global_v4_if(const void* ptr, bool pred) {
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    asm volatile("{\n .reg .pred q;\n setp.ne.b32 q, %5, 0;\n @q ld.global.v4.b32 {%0, %1, %2, %3}, [%4];\n}"
                 : "+r"(v.x), "+r"(v.y), "+r"(v.z), "+r"(v.w) : "l"(ptr), "r"((uint32_t)pred) : "memory");
    return v;
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// The loaded registers only hold their values once the wait above has run, but to the compiler they were defined by
// the load statement: nothing stops it from moving an instruction that reads them above the wait.  Passing them
// through an (empty) volatile statement placed after the wait makes every later use depend on that statement.
__device__ __forceinline__ void tmem_regs_ready(uint32_t (&r)[64]) {
    asm volatile("" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31]));
    asm volatile("" : "+r"(r[32]), "+r"(r[33]), "+r"(r[34]), "+r"(r[35]), "+r"(r[36]), "+r"(r[37]), "+r"(r[38]), "+r"(r[39]), "+r"(r[40]), "+r"(r[41]), "+r"(r[42]), "+r"(r[43]), "+r"(r[44]), "+r"(r[45]), "+r"(r[46]), "+r"(r[47]), "+r"(r[48]), "+r"(r[49]), "+r"(r[50]), "+r"(r[51]), "+r"(r[52]), "+r"(r[53]), "+r"(r[54]), "+r"(r[55]), "+r"(r[56]), "+r"(r[57]), "+r"(r[58]), "+r"(r[59]), "+r"(r[60]), "+r"(r[61]), "+r"(r[62]), "+r"(r[63]));
}

// Shared-memory matrix descriptor, SWIZZLE_128B, descriptor version 1 (sm_100).
//   K-major : rows of 128 B (64 bf16 along K); 8-row groups every `sbo` bytes.
//   MN-major: rows of 128 B (64 bf16 along M/N), one row per k; 8-k groups every `sbo` bytes,
//             the next 64-element chunk along M/N every `lbo` bytes.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// Stored coordinates (r, c) of an operand -> the first four coordinates of its tensor map (the fifth is the problem of a batch).
// FULL = false: the instantiation for plain calls (no page-interleaved operand, no batch, no alpha / beta, no operand split
// along K) leaves those branches out -- 0.5-0.7 us on a 15-30 us GEMM, 0.5 % on the large ones.
template <bool FULL = true>
__device__ __forceinline__ void to_coords(const OpMap& o, int r, int c, int& x, int& y, int& z, int& u) {
    int g, rr, xx;                                   // strip, row inside the strip, column inside the strip row
    if (o.split == 2) { o.w.divmod(c, g, xx); rr = r; }
    else if (o.split == 1) { o.h.divmod(r, g, rr); xx = c; }
    else { g = 0; rr = r; xx = c; }
    if (FULL && o.il_mode == 1) { o.il_kr.divmod(rr, u, y); x = xx; z = g; }
    else if (FULL && o.il_mode == 2) { o.il_sc.divmod(xx, y, x); z = rr; u = g; }
    else { x = xx; y = rr; z = g; u = 0; }
}
// il_mode 3: the 128-byte line of the buffer that holds the 64 elements from stored (r, c) on, c a multiple of 64; a piece
// outside the matrix gets a line past the end of the tensor map, which the copy engine fills with zeros.
__device__ __forceinline__ int line_of(const OpMap& o, int r, int c) {
    if (r >= o.rows || c >= o.cols) return o.lines;
    int g = 0, rr = r, xx = c;
    if (o.split == 2) o.w.divmod(c, g, xx);
    else if (o.split == 1) o.h.divmod(r, g, rr);
    const int e = rr * o.roww + xx;                  // element of the strip's packed contents (< 2^31: checked on the host)
    int j, x;
    o.il_sc.divmod(e, j, x);
    return (int)((((int64_t)j * o.nstrips + g) * (int64_t)o.il_sc.d + x) >> 6);
}
// Element offset of C[m][n] in its buffer (any layout).
template <bool FULL = true>
__device__ __forceinline__ int64_t c_offset(const GemmParams& p, int64_t m, int64_t n) {
    // (multiply-shift divisions only: a 64-bit division is a subroutine of several hundred cycles)
    int g = 0, rr = (int)m, xx = (int)n;             // strip, row inside the strip, column inside the strip row
    if (p.c.split == 2) p.c.w.divmod((int)n, g, xx);
    else if (p.c.split == 1) p.c.h.divmod((int)m, g, rr);
    if (FULL && p.c.il_mode == 1) {                  // a chunk holds il_kr whole strip rows
        int j, y;
        p.c.il_kr.divmod(rr, j, y);
        return ((int64_t)j * p.c_nstrips + g) * p.c_ichunk + (int64_t)y * p.c_row + xx;
    }
    if (FULL && p.c.il_mode == 3) {                  // chunks and strip rows do not line up: the general form
        int j, x;
        p.c.il_sc.divmod(rr * p.c.roww + xx, j, x);
        return ((int64_t)j * p.c_nstrips + g) * p.c_ichunk + x;
    }
    if (FULL && p.c.il_mode == 2) {                  // a strip row spans c_cpr whole chunks
        int cj, x;
        p.c.il_sc.divmod(xx, cj, x);
        return (((int64_t)rr * p.c_cpr + cj) * p.c_nstrips + g) * p.c_ichunk + x;
    }
    if (FULL && p.c_wlast && g == p.c.nstrips - 1) return (int64_t)g * p.c_stride + (int64_t)rr * p.c_wlast + xx;   // a narrower last strip
    return (int64_t)g * p.c_stride + (int64_t)rr * p.c_row + xx;
}

// Ragged K: first row, k blocks and rows of the last block of problem e (an empty or out-of-range problem: one block of
// zero rows, so that its output is written as zeros).
__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

struct KRange { int k0, nkb, rem; };
__device__ __forceinline__ KRange k_range(const int32_t* k_offs, int e, int Ktot) {
    const int o0 = __ldg(k_offs + e), o1 = __ldg(k_offs + e + 1);
    KRange r;
    if (o0 < 0 || o1 > Ktot || o1 < o0) { atomicExch(&g_gemm_status, 5); r.k0 = 0; r.nkb = 1; r.rem = 0; return r; }
    const int cnt = o1 - o0;
    r.k0 = o0; r.nkb = cnt > 0 ? (cnt + BK - 1) / BK : 1; r.rem = cnt - (r.nkb - 1) * BK;
    return r;
}

// e: problem of the batch; skip: an empty tile of a ragged batch.  Balanced split: the unit computes k blocks [kb0, kb1) of
// the tile; part = 0: all of them (a plain tile), 1: a share -- the tile is split among `nshare` consecutive units, of
// which this one is number `mine` (0 holds k = 0); every sharer writes its partial sums to its slot of the workspace and
// then reduces and stores every nshare-th 64-column piece of the tile.
struct TileCoord { int m0, m1, n0, n1, split, e; bool skip; int kb0, kb1, part, nshare, mine, round; };   // round: of whole tiles (-1: a share)

// Tiles of this CTA (pair).  The schedulable units (CTAs, or CTA pairs) serve `groups` strip ranges
// (chiplet-grouped raster): group g owns the tiles of strip range g and walks them in panels of
// `panel` m-tiles (m fastest inside a panel, then n, then the next panel).
// Every group gets the SAME number of units (upg = units / groups) so that the groups advance in
// lockstep through the same m-panels and share the A operand in L2; the units left over ("floaters")
// and, at the end, everybody work through a pool made of the last few tiles of every group:
//   grouped unit : rounds [0, R) -> tile (index + round * upg) of its own group, then the pool
//   floater f    : rounds [0, R) -> pool entries f, f + F, ...,                  then the pool
// with R = min(total / units, per_group / upg); pool entries alternate between the groups.
// The per-launch constants (units, upg, floaters, R, pool size) come from the host; tiles x splits < 2^31.
struct Scheduler {
    const GemmParams& p;
    int gm, gn;                     // tile grid of one group
    int unit, units, upg, floaters, my_g, idx, bm, bn, rounds, pool_per_group;
    const int* rag;                 // ragged batch, dense walk: rag[e] = m-tiles of the problems before e (shared memory)
    __device__ Scheduler(const GemmParams& p_, int unit_, int bm_, int bn_, const int* rag_) : p(p_), unit(unit_), bm(bm_), bn(bn_), rag(rag_) {
        gm = p.sch_gm; gn = p.sch_gn; units = p.sch_units; upg = p.sch_upg; floaters = p.sch_floaters;
        rounds = p.sch_rounds; pool_per_group = p.sch_pool_per_group;
        my_g = unit < upg * p.groups ? p.fd_upg.div(unit) : -1;  // -1: floater
        idx = my_g >= 0 ? unit - my_g * upg : unit - upg * p.groups;
    }
    // Ragged batch: tile q of the walk (n fastest, then the m-tiles of problem 0, 1, ...) by a search in the prefix.
    __device__ bool get_ragged(int it, TileCoord& t) const {
        const int E = p.batch, q = unit + it * units;
        if (q >= rag[E] * p.tiles_n) return false;
        int mt, tn;
        p.fd_tiles_n.divmod(q, mt, tn);
        int lo = 0, hi = E;                              // the last problem whose prefix is <= mt (empty problems share a prefix)
        while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (rag[mid] <= mt) lo = mid; else hi = mid; }
        const int o0 = __ldg(p.m_offs + lo), o1 = __ldg(p.m_offs + lo + 1);
        int sn, jn;
        p.fd_tps_n.divmod(tn, sn, jn);
        t.e = lo; t.split = 0; t.skip = false; t.part = 0; t.round = it;
        t.m0 = o0 + (mt - rag[lo]) * bm; t.m1 = min(t.m0 + bm, o1);
        t.n0 = sn * p.Wn + jn * bn; t.n1 = min(t.n0 + bn, (sn + 1) * p.Wn);
        return true;
    }
    // Balanced split.  A group's tiles that do not fill a whole round of its units -- the first bal_tiles tiles of its walk --
    // are laid end to end along K and cut into equal shares of k blocks, one per unit (the first bal_units units; share of
    // unit u = [lo(u), lo(u + 1)), lo(u) = u * q + min(u, r)): every unit starts with its share, then walks whole tiles
    // round by round like everybody else.  A tile of the first kind is thus split among consecutive units; each of them
    // hands its partial sums to the others through the workspace and reduces its part of the tile's columns (epilogue
    // warps only: the tensor cores are on the unit's next tile by then).
    __device__ int bal_lo(int u) const { u = min(u, p.bal_units); return u * p.bal_q + min(u, p.bal_r); }
    template <bool FULL>
    __device__ bool get_balanced(int it, TileCoord& t) const {
        if (my_g < 0) return false;
        const int nkb = p.num_kb, lo = bal_lo(idx), hi = bal_lo(idx + 1);
        const int first = p.fd_num_kb.div(lo), shares = hi > lo ? p.fd_num_kb.div(hi - 1) - first + 1 : 0;
        t.split = 0; t.e = 0; t.skip = false; t.nshare = 1; t.mine = 0;
        if (it < shares) {
            const int tile = first + it, k0 = tile * nkb;
            t.kb0 = max(lo, k0) - k0; t.kb1 = min(hi, k0 + nkb) - k0;
            t.part = (t.kb0 > 0 || t.kb1 < nkb) ? 1 : 0;
            t.round = -1;
            if (t.part) {                                  // the units whose shares meet this tile: u0 holds k0, the last one k0 + nkb - 1
                int u0 = idx;
                while (bal_lo(u0) > k0) --u0;
                int u1 = idx;
                while (bal_lo(u1 + 1) < k0 + nkb) ++u1;
                t.mine = idx - u0; t.nshare = u1 - u0 + 1;
            }
            coords<FULL>(my_g, tile, t);
            return true;
        }
        const int tile = p.bal_tiles + idx + (it - shares) * upg;
        if (tile >= p.sch_per_group) return false;
        t.kb0 = 0; t.kb1 = nkb; t.part = 0; t.round = it - shares;
        coords<FULL>(my_g, tile, t);
        return true;
    }
    // tile i of group g's walk -> its rows and columns
    template <bool FULL>
    __device__ void coords(int g, int i, TileCoord& t) const {
        int pn, rem;
        p.fd_per_panel.divmod(i, pn, rem);
        const bool tail = gm - pn * p.panel < p.panel;   // the last panel may be lower
        const int ph = tail ? gm - pn * p.panel : p.panel;
        int ln, lr;
        if (tail) { ln = rem / ph; lr = rem - ln * ph; } else p.fd_panel.divmod(rem, ln, lr);
        int lm = pn * p.panel + lr;
        int tm = lm + (p.group_dim == 1 ? g * gm : 0), tn = ln + (p.group_dim == 0 && p.groups > 1 ? g * gn : 0);
        if (FULL && p.group_dim == 2) { int qm, qn; p.fd_groups_n.divmod(g, qm, qn); tm += qm * gm; tn += qn * gn; }
        int sm, jm, sn, jn;
        p.fd_tps_m.divmod(tm, sm, jm);
        p.fd_tps_n.divmod(tn, sn, jn);
        t.m0 = sm * p.Wm + jm * bm; t.m1 = min(t.m0 + bm, (sm + 1) * p.Wm);
        t.n0 = sn * p.Wn + jn * bn; t.n1 = min(t.n0 + bn, (sn + 1) * p.Wn);
        if (FULL) { t.m1 = min(t.m1, p.M); t.n1 = min(t.n1, p.N); }     // (a last strip that is lower / narrower than the others)
    }
    template <int RAG, bool FULL>
    __device__ bool get(int it, TileCoord& t) const {
        if (RAG == 1 && rag) return get_ragged(it, t);
        if (RAG == 0 && p.bal) return get_balanced<FULL>(it, t);
        t.part = 0; t.round = it;
        if (RAG == 0 && p.ks) {                           // cluster split: unit = cluster, one tile each
            if (it > 0) return false;
            int g = 0, i = unit;
            if (p.groups > 1) { g = unit / p.sch_per_group; i = unit - g * p.sch_per_group; }
            t.split = 0; t.e = 0; t.skip = false;
            coords<FULL>(g, i, t);
            return true;
        }
        int g, i;
        if (it < rounds && my_g >= 0) { g = my_g; i = idx + it * upg; }
        else {
            const int q = it < rounds ? idx + it * floaters : floaters * rounds + unit + (it - rounds) * units;
            int j = q;
            g = 0;
            if (p.groups > 1) p.fd_groups.divmod(q, j, g);
            if (j >= pool_per_group) return false;
            i = rounds * upg + j;
        }
        t.split = 0;
        if (p.splits > 1) { int ii; p.fd_splits.divmod(i, ii, t.split); i = ii; }   // the splits of one tile are neighbours in the walk
        t.e = 0;
        if (FULL && p.batch > 1) { int ii; p.fd_tiles_per_problem.divmod(i, t.e, ii); i = ii; }
        coords<FULL>(g, i, t);
        t.skip = FULL && RAG == 0 && (t.m0 >= p.M || t.n0 >= p.N);   // the tile grid of a shorter last strip has empty places
        if (RAG == 1 && p.m_offs) {                      // rows of this problem inside the concatenated A and C
            const int o0 = __ldg(p.m_offs + t.e), o1 = __ldg(p.m_offs + t.e + 1);
            const bool bad = o0 < 0 || o1 > p.M || o1 - o0 > p.Wm;   // outside A / C, or more rows than the caller's bound:
            if (bad && t.m0 == 0 && t.n0 == 0) atomicExch(&g_gemm_status, 5);   // reported, and the problem is left out
            t.skip = bad || t.m0 >= o1 - o0;
            t.m0 += o0; t.m1 = min(t.m0 + bm, o1);
        }
        return true;
    }
};

// RAG: 1 = ragged M (ccl_gemm_grouped), 2 = ragged K (ccl_gemm_grouped_k) -- instantiations of their own, so that the tile
// walk and the k loops of all other calls stay as they are (the extra branches cost 1-1.5 us on a 15-30 us GEMM)
// KS > 0: cluster split along K (CTAS = 1): the KS CTAs of a cluster share one tile
template <int BN, int CTAS, bool SWIGLU = false, int RAG = 0, bool FULL = true, int KS = 0>
__global__ void __launch_bounds__(kGemmThreads, 1)
ccl_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                const __grid_constant__ CUtensorMap map_c, const __grid_constant__ CUtensorMap map_a2,
                const __grid_constant__ CUtensorMap map_b2, const __grid_constant__ CUtensorMap map_c2,
                const __grid_constant__ GemmParams gp) {
    // map_a2 / map_b2 / map_c2: the last strip of an operand whose strips are not all alike (OpMap::rag); copies of the
    // first three otherwise
    // The parameters are read from shared memory: the threads fetch the block's words side by side, so
    // the cold constant-cache misses at kernel start overlap instead of queueing up in every role's set-up.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel's CTAs may be placed as SMs free up
    __shared__ GemmParams p;
    {
        static_assert(sizeof(GemmParams) % 4 == 0, "GemmParams is copied word by word");
        const uint32_t* src = reinterpret_cast<const uint32_t*>(&gp);
        uint32_t* dst = reinterpret_cast<uint32_t*>(&p);
        for (int i = threadIdx.x; i < (int)(sizeof(GemmParams) / 4); i += kGemmThreads) dst[i] = src[i];
    }
    // A tile wider than 256 columns is computed as two sub-tiles (one MMA each per k step), the first 256 columns wide,
    // the second the rest (256 or 128), each with a 256-column half of TMEM; narrower tiles use the two halves as a
    // double buffer.
    static_assert(BN <= 256 || BN == 384 || BN == 512, "tile widths");
    constexpr int NSUB = BN > 256 ? 2 : 1;
    constexpr int SUBN = NSUB == 1 ? BN : 256;        // width of the first sub-tile = columns from one sub-tile to the next
    constexpr int SUBN1 = NSUB == 1 ? 0 : BN - 256;   // width of the second
    constexpr int ACC_COLS = 256;                     // TMEM columns between accumulators
    constexpr int NACC = 2;                           // accumulator barriers in use
    static_assert(!SWIGLU || BN == 512, "the gated activation pairs the two accumulators of a wide tile");
    constexpr int TILE_N = SWIGLU ? SUBN : BN;        // tile width in the columns the tile walk counts (output columns)
    constexpr int SUBH = SUBN / CTAS;                // B columns of the first sub-tile this CTA stages
    constexpr int SUBH1 = SUBN1 / CTAS;              // ... of the second
    static_assert(BN != 384 || CTAS == 2, "the 384-wide tile is a CTA-pair tile");
    // B boxes are 64 columns wide for an N-contiguous B; a K-contiguous B is staged in one box per sub-tile, except in
    // the 384-wide tile, whose sub-tiles differ in width: 64-row boxes there (same place in shared memory either way)
    constexpr bool B64 = BN == 384;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* epi = smem + (size_t)gp.stages * gp.stage_bytes;     // 1024-byte aligned: stage sizes are multiples of 1 KB
    uint64_t* bars = reinterpret_cast<uint64_t*>(epi + kEpiBytes);
    uint64_t* full = bars;                           // used in the leader CTA only
    uint64_t* empty = bars + gp.stages;               // one set per CTA
    uint64_t* tmem_full = bars + 2 * gp.stages;       // one set per CTA
    uint64_t* tmem_empty = tmem_full + 4;            // used in the leader CTA only
    uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(tmem_empty + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = CTAS == 2 ? cluster_ctarank() : 0;
    const bool leader = rank == 0;
    static_assert(KS == 0 || (CTAS == 1 && BN <= 256 && !SWIGLU && RAG == 0 && !FULL), "the cluster split is a plain 1-CTA-per-tile kernel");
    const uint32_t krank = KS ? cluster_ctarank() : 0;   // cluster split: which part of K this CTA computes

    if (threadIdx.x == 0) {
        prefetch_tmap(&map_a);
        prefetch_tmap(&map_b);
        prefetch_tmap(&map_c);
        for (int s = 0; s < gp.stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int a = 0; a < NACC; ++a) { mbar_init(&tmem_full[a], 1); mbar_init(&tmem_empty[a], kEpiWarps * CTAS); }
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc<CTAS>(tmem_ptr, kTmemCols);
    tc_fence_before();
    __syncthreads();
    if (CTAS == 2) cluster_sync();                   // the peer's barriers exist before anything remote touches them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr;
    // Everything before the dependency wait overlaps the previous kernel's tail.  A ragged batch reads its offsets from
    // global memory right away and waits here; otherwise every role waits where it first needs global memory -- the
    // producer only after it has worked out its first tile's coordinates.
    if (RAG != 0) asm volatile("griddepcontrol.wait;" ::: "memory");

    // Ragged batch with a dense walk: m-tiles of every problem, as an exclusive prefix over the problems.
    int* rag_prefix = nullptr;
    if (RAG == 1 && p.rag_dense) {
        int* part = reinterpret_cast<int*>(tmem_ptr + 4);           // one partial sum per thread, then the prefix itself
        rag_prefix = part + kGemmThreads;
        const int E = p.batch, bm = BM * CTAS, per = (E + kGemmThreads - 1) / kGemmThreads;
        const int lo = min(E, (int)threadIdx.x * per), hi = min(E, lo + per);
        auto tiles_of = [&](int e) {
            const int o0 = __ldg(p.m_offs + e), o1 = __ldg(p.m_offs + e + 1);
            if (o0 < 0 || o1 > p.M || o1 - o0 > p.Wm) { atomicExch(&g_gemm_status, 5); return 0; }   // reported, left out
            return o1 > o0 ? (o1 - o0 + bm - 1) / bm : 0;
        };
        int sum = 0;
        for (int e = lo; e < hi; ++e) sum += tiles_of(e);
        part[threadIdx.x] = sum;
        __syncthreads();
        if (threadIdx.x == 0) {
            int run = 0;
            for (int i = 0; i < kGemmThreads; ++i) { const int v = part[i]; part[i] = run; run += v; }
            rag_prefix[E] = run;
        }
        __syncthreads();
        int run = part[threadIdx.x];
        for (int e = lo; e < hi; ++e) { rag_prefix[e] = run; run += tiles_of(e); }
        __syncthreads();
    }
    Scheduler sched(p, (int)(blockIdx.x / (KS ? KS : CTAS)), BM * CTAS, TILE_N, rag_prefix);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        // One lane per TMA box of a stage (at most 6): the whole warp walks the tile/k loop, every lane
        // polls the stage's "empty" barrier, lane 0 posts the byte count and each active lane issues its
        // own box, so a stage is refilled in one issue slot instead of a serial chain.
        // 64-wide boxes per MN-major A tile / B sub-tile.  (The 96 columns a CTA of a 256 x 192 pair tile stages of an
        // N-contiguous B are fetched as two boxes, the second of which is half used: what it holds beyond the 96th
        // column -- the peer's columns, the next tile's, or the zero fill past the strip's end -- is never read.)
        constexpr int NA = BM / 64, NC = (SUBH + 63) / 64, NC1 = (SUBH1 + 63) / 64;
        const bool b64 = B64 || p.b_mn;
        const int nA = p.a_mn ? NA : 1;
        const int nB = b64 ? NC + NC1 : NSUB;
        const bool active = lane < nA + nB;
        const bool isA = lane < nA;
        const int bi = isA ? lane : lane - nA;                // box index within its operand
        const CUtensorMap* map = isA ? &map_a : &map_b;
        const OpMap om = isA ? p.a : p.b;
        const bool mn = isA ? p.a_mn != 0 : p.b_mn != 0;
        // K runs along the tensor map's x for a K-contiguous operand and along y otherwise; unless the
        // operand is split along K itself (rare) only that coordinate changes from one k block to the next
        // (a page-interleaved operand recomputes its coordinates every k block as well)
        const bool ksplit = FULL && ((mn ? om.split == 1 : om.split == 2) || om.il_mode != 0);
        const bool gather_a = FULL && p.a.il_mode == 3, gather_b = FULL && p.b.il_mode == 3;
        const bool box = active && !(isA ? gather_a : gather_b);     // this lane issues one box per stage
        uint32_t soff;                                        // byte offset of the box inside a stage
        int off;                                              // offset of the box along M (A) or N (B) from the tile origin
        int hsel = 0;                                         // sub-tile of a B box
        if (isA) { soff = mn ? (uint32_t)bi * (64 * BK * 2) : 0u; off = (int)rank * BM + (mn ? 64 * bi : 0); }
        else if (b64) { const int h = bi >= NC ? 1 : 0, c = bi - h * NC; hsel = h; soff = p.a_bytes + (uint32_t)(h * SUBH * BK * 2 + c * 64 * BK * 2); off = h * SUBN + (int)rank * (h ? SUBH1 : SUBH) + 64 * c; }
        else { hsel = bi; soff = p.a_bytes + (uint32_t)(bi * SUBH * BK * 2); off = bi * SUBN + (int)rank * SUBH; }
        if (SWIGLU && !isA) off -= hsel * SUBN;               // sub-tile 1 is not 256 columns on but pair_dist (below)
        const uint32_t full0 = CTAS == 2 ? map_to_cta(smem_u32(&full[0]), 0) : smem_u32(&full[0]);
        int stage = 0;
        uint32_t phase = 0;
        TileCoord t;
        bool ok = true;
        // loop constants in registers (the asm statements below are memory barriers to the compiler)
        const int stages = p.stages, num_kb = p.num_kb, kbps = p.kb_per_split;
        const uint32_t stage_bytes = p.stage_bytes, tx_bytes = p.tx_bytes;
        const bool post_tx = lane == 0 && leader;
        bool dep_pending = RAG == 0;                          // the previous kernel has not been waited for yet
        for (int it = 0; ok && sched.template get<RAG, FULL>(it, t); ++it) {
            if (t.skip) continue;
            if (KS) t.split = (int)krank;
            if (p.wave_ctr && t.round >= 1 && t.round < p.sch_rounds && t.round % p.wave_period == 0) {   // wait (bounded) until every CTA has issued its previous tiles
                if (lane == 0) {
                    atomicAdd(p.wave_ctr, 1u);
                    const unsigned int target = gridDim.x * (unsigned int)(t.round / p.wave_period);
                    const uint64_t t0 = global_timer_ns();
                    while (ld_acquire_u32(p.wave_ctr) < target && global_timer_ns() - t0 < (uint64_t)p.wave_wait_ns) { }
                }
                __syncwarp();
            }
            int base = (isA ? t.m0 : t.n0) + off;
            // output column n0 of strip g -> B column n0 + g * pair_dist (gate) and one pair_dist further (up)
            if (SWIGLU && !isA) base += (p.fd_wn.div(t.n0) + hsel) * p.pair_dist;
            int x, y, z, u;
            if (mn) to_coords<FULL>(om, 0, base, x, y, z, u); else to_coords<FULL>(om, base, 0, x, y, z, u);
            const CUtensorMap* mp = map;
            if (FULL && om.rag && z == om.nstrips - 1) { mp = isA ? &map_a2 : &map_b2; z = 0; }
            int kb0 = t.split * kbps, kb1 = min(num_kb, kb0 + kbps), kbase = 0;
            if (RAG == 0 && p.bal) { kb0 = t.kb0; kb1 = t.kb1; }
            if (RAG == 2) { const KRange kr = k_range(p.k_offs, t.e, p.K); kb0 = 0; kb1 = kr.nkb; kbase = kr.k0; }
            if (dep_pending) { asm volatile("griddepcontrol.wait;" ::: "memory"); dep_pending = false; }   // the first operand load is next
            for (int kb = kb0; kb < kb1; ++kb) {
                ok = mbar_wait_bounded(&empty[stage], phase ^ 1);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) { if (lane == 0) atomicExch(&g_gemm_status, 1); break; }
                // (the byte count may be posted after a copy has completed: the phase cannot end before this arrival)
                if (post_tx) mbar_expect_tx(&full[stage], tx_bytes * CTAS);
                const int k0 = kbase + kb * BK;
                if (ksplit) { if (mn) to_coords<FULL>(om, k0, base, x, y, z, u); else to_coords<FULL>(om, base, k0, x, y, z, u); }
                else if (mn) y = k0; else x = k0;
                if (box) tma_load<CTAS>(smem + (size_t)stage * stage_bytes + soff, mp, full0 + (uint32_t)stage * 8u, x, y, z, u, t.e * om.batched);
                if (FULL && (gather_a || gather_b)) {
                    // An operand whose chunks and strip rows do not line up: its part of the stage is fetched as single
                    // 128-byte rows (the swizzle is a function of the shared-memory address, so the rows land exactly
                    // where a box would have put them), the 32 lanes taking turns.
                    unsigned char* st0 = smem + (size_t)stage * stage_bytes;
                    const uint32_t bar = full0 + (uint32_t)stage * 8u;
                    if (gather_a)
                        for (int i = lane; i < BM; i += 32) {
                            int r, c; uint32_t so;
                            if (p.a_mn) { const int ch = i >> 6, kr = i & 63; r = k0 + kr; c = t.m0 + (int)rank * BM + 64 * ch; so = (uint32_t)(ch * 64 * BK * 2 + kr * 128); }
                            else { r = t.m0 + (int)rank * BM + i; c = k0; so = (uint32_t)i * 128u; }
                            tma_load<CTAS>(st0 + so, &map_a, bar, 0, line_of(p.a, r, c), 0, 0, 0);
                        }
                    if (gather_b)
                        for (int i = lane; i < SUBH + SUBH1; i += 32) {
                            int r, c; uint32_t so;
                            if (p.b_mn) {
                                const int ch = i >> 6, kr = i & 63, h = ch >= NC ? 1 : 0, cc = ch - h * NC;
                                r = k0 + kr; c = t.n0 + h * SUBN + (int)rank * (h ? SUBH1 : SUBH) + 64 * cc;
                                so = p.a_bytes + (uint32_t)(h * SUBH * BK * 2 + cc * 64 * BK * 2 + kr * 128);
                            } else {
                                const int h = i >= SUBH ? 1 : 0, rr = i - h * SUBH;
                                r = t.n0 + h * SUBN + (int)rank * (h ? SUBH1 : SUBH) + rr; c = k0;
                                so = p.a_bytes + (uint32_t)(h * SUBH * BK * 2 + rr * 128);
                            }
                            tma_load<CTAS>(st0 + so, &map_b, bar, 0, line_of(p.b, r, c), 0, 0, 0);
                        }
                }
                if (++stage == stages) { stage = 0; phase ^= 1; }
            }
        }
        if (KS) { __syncwarp(); cluster_sync(); cluster_sync(); }   // the two meetings of the cluster split (see the epilogue)
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (RAG == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
        // The whole warp runs the loop with the same values in every lane and one elected lane issues the tcgen05
        // instructions: values the compiler can prove warp-uniform (kernel parameters, shuffles, votes) live in uniform
        // registers, which is where the MMA takes its descriptors from -- a single diverged lane had to move every
        // operand across for every instruction.
        if (leader) {
            const uint32_t FULLMASK = 0xffffffffu;
            int stage = 0;
            uint32_t phase = 0;
            TileCoord t;
            bool ok = true;
            const uint32_t a_lbo = gp.a_mn ? 64 * BK * 2 : 16, b_lbo = gp.b_mn ? 64 * BK * 2 : 16;
            const uint32_t a_kstep = gp.a_mn ? (16 * 128) >> 4 : (16 * 2) >> 4;     // descriptor units (16 B) per UMMA_K = 16
            const uint32_t b_kstep = gp.b_mn ? (16 * 128) >> 4 : (16 * 2) >> 4;
            const int stages = gp.stages, num_kb = gp.num_kb, kbps = gp.kb_per_split;
            const uint32_t stage_bytes = gp.stage_bytes, a_bytes = gp.a_bytes, idesc = gp.idesc, smem0 = smem_u32(smem);
            const uint32_t tmem_b = __shfl_sync(FULLMASK, tmem_base, 0);
            int done = 0;                                   // tiles computed so far (empty tiles of a ragged batch do not count)
            bool ready = false;
            // running values of the current stage: descriptor low words (the address field counts 16-byte units; a stage
            // is a multiple of 1 KB), the shared-memory addresses of its two barriers
            const uint64_t adesc0 = smem_desc(smem0, a_lbo, 1024), bdesc0 = smem_desc(smem0 + a_bytes, b_lbo, 1024);
            const uint32_t a_hi = (uint32_t)(adesc0 >> 32), b_hi = (uint32_t)(bdesc0 >> 32), a_lo0 = (uint32_t)adesc0, b_lo0 = (uint32_t)bdesc0;
            const uint32_t st_units = stage_bytes >> 4, fbar0 = smem_u32(&full[0]), ebar0 = smem_u32(&empty[0]);
            uint32_t a_lo = a_lo0, b_lo = b_lo0, fbar = fbar0, ebar = ebar0;
            for (int it = 0; ok; ++it) {
                const bool more = sched.template get<RAG, FULL>(it, t);
                if (!__shfl_sync(FULLMASK, (int)more, 0)) break;
                if ((RAG != 0 || FULL) && __shfl_sync(FULLMASK, (int)t.skip, 0)) continue;
                if (KS) t.split = (int)krank;
                // NSUB == 1: TMEM half (done & 1) is this tile's accumulator, the other half is being drained.
                // NSUB == 2: both halves belong to this tile; half h may be overwritten once the epilogue
                //            of the previous tile has drained it.
                const int acc0 = NSUB == 1 ? (done & 1) : 0;
                const uint32_t acc_phase = NSUB == 1 ? ((uint32_t)(done >> 1) & 1) : ((uint32_t)done & 1);
                ++done;
                int kb0 = t.split * kbps, kb1 = min(num_kb, kb0 + kbps), tail = BK;
                if (RAG == 0 && gp.bal) { kb0 = t.kb0; kb1 = t.kb1; }
                if (RAG == 2) { const KRange kr = k_range(p.k_offs, t.e, p.K); kb0 = 0; kb1 = kr.nkb; tail = kr.rem; }
                kb0 = __shfl_sync(FULLMASK, kb0, 0); kb1 = __shfl_sync(FULLMASK, kb1, 0);
                if (RAG == 2) tail = __shfl_sync(FULLMASK, tail, 0);
                for (int kb = kb0; ok && kb < kb1; ++kb) {
                    // (the copies' completion on the barrier orders the operand bytes before the MMAs that read them;
                    // tcgen05 fences are only needed around the accumulator hand-over below)
                    // `ready`: this stage's barrier was already seen complete by the look-ahead of the previous k block
                    if (!ready) {
                        ok = __all_sync(FULLMASK, mbar_wait_bounded_addr(fbar, phase));
                        if (!ok) { if (lane == 0) atomicExch(&g_gemm_status, 3); break; }
                    }
                    // the stage after this one (its barrier is looked at while this block's MMAs are issued)
                    uint32_t n_a_lo = a_lo + st_units, n_b_lo = b_lo + st_units, n_fbar = fbar + 8, n_ebar = ebar + 8, n_phase = phase;
                    if (++stage == stages) { stage = 0; n_a_lo = a_lo0; n_b_lo = b_lo0; n_fbar = fbar0; n_ebar = ebar0; n_phase = phase ^ 1; }
                    // Ragged K, last block of a problem: only the 16-row k steps that hold rows of this problem are
                    // issued, and the rows of the last step that belong to the next problem are zeroed in shared memory
                    // (both operands are [k][64 columns] boxes of 128-byte rows here, so a k row is a whole line).
                    const bool cut = RAG == 2 && tail < BK && kb == kb1 - 1;
                    int ksteps = BK / 16;
                    if (cut) {
                        ksteps = tail > 0 ? (tail + 15) / 16 : 1;
                        const uint32_t sa = (a_lo & 0x3FFFu) << 4;          // the stage's shared-memory address, back from the descriptor
                        const int nboxes = (int)(stage_bytes / (64 * BK * 2));
                        for (int i = tail * nboxes + lane; i < ksteps * 16 * nboxes; i += 32) {     // the lanes share the (row, box) pairs
                            const int r = i / nboxes, b = i - r * nboxes;
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(sa + (uint32_t)(b * 64 * BK * 2 + r * 128 + c * 16)), "r"(0u) : "memory");
                        }
                        fence_proxy_async();
                        __syncwarp();
                    }
                    ready = false;
#pragma unroll
                    for (int h = 0; h < NSUB; ++h) {
                        if (kb == kb0) {
                            ok = __all_sync(FULLMASK, mbar_wait_bounded(&tmem_empty[acc0 + h], acc_phase ^ 1));
                            if (!ok) { if (lane == 0) atomicExch(&g_gemm_status, 2); break; }
                            tc_fence_after();
                        }
                        const uint32_t tmem_d = tmem_b + (uint32_t)((acc0 + h) * ACC_COLS);
                        const uint32_t b_lo_h = b_lo + (uint32_t)(h * ((SUBH * BK * 2) >> 4));
                        // (the instruction descriptor carries the width of the first sub-tile: N >> 3 in bits 17-22)
                        const uint32_t idesc_h = (NSUB == 2 && SUBN1 != SUBN && h == 1) ? (idesc & ~(0x3Fu << 17)) | ((uint32_t)(SUBN1 >> 3) << 17) : idesc;
                        if (!cut) {                           // (the common path: four back-to-back MMAs and a look at the next stage's barrier)
                            static_assert(BK / 16 == 4, "four MMAs per k block");
                            if (h == 0) ready = __all_sync(FULLMASK, umma_bf16_x4<CTAS, true>(tmem_d, a_lo, a_hi, b_lo_h, b_hi, a_kstep, b_kstep, idesc_h, kb != kb0, n_fbar, n_phase) != 0);
                            else umma_bf16_x4<CTAS, false>(tmem_d, a_lo, a_hi, b_lo_h, b_hi, a_kstep, b_kstep, idesc_h, kb != kb0, 0u, 0u);
                        } else {
                            const uint64_t adesc = ((uint64_t)a_hi << 32) | a_lo, bdesc = ((uint64_t)b_hi << 32) | b_lo_h;
                            if (lane == 0) {
#pragma unroll 1
                                for (int k = 0; k < ksteps; ++k)
                                    umma_bf16<CTAS>(tmem_d, adesc + (uint64_t)(k * a_kstep), bdesc + (uint64_t)(k * b_kstep), idesc_h, ((kb - kb0) | k) != 0);
                            }
                            __syncwarp();
                        }
                    }
                    if (!ok) break;
                    umma_commit_addr<CTAS>(ebar);              // frees the stage (in both CTAs) once these MMAs have read it
                    a_lo = n_a_lo; b_lo = n_b_lo; fbar = n_fbar; ebar = n_ebar; phase = n_phase;
                }
                if (ok) umma_commit_addr<CTAS>(smem_u32(&tmem_full[acc0]));   // accumulator(s) complete (both CTAs); the sub-tiles of a wide tile finish together
            }
        }
        if (KS) { __syncwarp(); cluster_sync(); cluster_sync(); }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        if (RAG == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
        const int quad = warp & 3;                       // TMEM lane quadrant this warp may read
        constexpr int EW = kEpiWarps / 4;                // warps per quadrant
        const int hf = (warp - 2) >> 2;                  // which of them this one is
        const uint32_t tmem_empty0 = CTAS == 2 ? map_to_cta(smem_u32(&tmem_empty[0]), 0) : smem_u32(&tmem_empty[0]);
        TileCoord t;
        bool alive = true;
        uint32_t epi_count = 0;                          // TMA-stored pieces so far (selects the staging buffer)
        int done = 0;                                    // tiles drained so far
        TileCoord pend[2];                               // balanced split: shares written but not yet reduced
        int npend = 0;
        for (int it = 0; alive && sched.template get<RAG, FULL>(it, t); ++it) {
          if (t.skip) continue;
          const int tile_no = done++;
          int m = t.m0 + (int)rank * BM + quad * 32 + lane;
#pragma unroll 1                                         // one copy of the (large) drain code: a short GEMM pays for every instruction-cache miss
          for (int h = 0; h < (SWIGLU ? 1 : NSUB); ++h) {
            const int acc = NSUB == 1 ? (tile_no & 1) : h;
            const uint32_t acc_phase = NSUB == 1 ? ((uint32_t)(tile_no >> 1) & 1) : ((uint32_t)tile_no & 1);
            int nb = t.n0 + h * SUBN;                    // first (output) column of this sub-tile
            bool ok = h > 0 || mbar_wait_bounded(&tmem_full[acc], acc_phase);   // one "full" barrier per tile
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {
                if (lane == 0) atomicExch(&g_gemm_status, 4);
                if (KS) { cluster_sync(); cluster_sync(); }        // the others are waiting at the cluster's meetings
                alive = false; break;
            }
            tc_fence_after();
            const bool bal = RAG == 0 && !SWIGLU && p.bal;
            bool released = false;                                 // the accumulator has been handed back already
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * ACC_COLS);
            // Full 32-row x 64-column pieces go through shared memory (128-byte swizzle) and a TMA tile store
            // addressed through C's own tensor map; ragged pieces (tile clipped by a strip or the matrix edge)
            // and split-K partial sums are stored from registers.
            int row0 = t.m0 + (int)rank * BM + quad * 32;
            bool rows_full = row0 + 32 <= t.m1;
            // C map coordinates of (row0, nb): a tile lies inside one strip, so only x moves from piece to piece
            // (unless a strip row is cut into chunks, which puts the chunk index in y as well)
            int cx0, cy0, cz0, cu0;
            to_coords<FULL>(p.c, row0, nb, cx0, cy0, cz0, cu0);
            const CUtensorMap* mpc = &map_c;
            if (FULL && p.c.rag && cz0 == p.c.nstrips - 1) { mpc = &map_c2; cz0 = 0; }
            const bool c_chunked = FULL && p.c.il_mode == 2;
            // One 64-column piece: registers -> C.  `r` holds 64 fp32 accumulators of this thread's row.
            // One 64-column piece of this warp's 32 rows -> C.  `pk` holds the piece already rounded to bf16 (two
            // values per word); full pieces go through shared memory and a TMA tile store, ragged ones are stored
            // from registers.  (The accumulator registers are packed right after the TMEM wait: nothing else reads
            // the registers a tcgen05.ld has written.)
            auto pack = [&](const uint32_t (&r)[64], uint32_t (&pk)[32]) {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
                    pk[i] = *reinterpret_cast<const uint32_t*>(&hh);
                }
            };
            auto store_packed = [&](const uint32_t (&pk)[32], int c) {
                const int n64 = nb + c * 64;
                if (rows_full && n64 + 64 <= t.n1 && !(FULL && p.c.il_mode == 3)) {
                    // staging: 32 KB in all -- two buffers per warp with four warps, one with eight
                    unsigned char* buf = epi + (size_t)(EW == 1 ? (warp - 2) * 2 + (epi_count & 1) : (warp - 2)) * (32 * 128);
                    if (epi_count >= 2 / EW) { if (lane == 0) tma_store_wait_read<2 / EW - 1>(); __syncwarp(); }   // buffer free again
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        *reinterpret_cast<uint4*>(buf + lane * 128 + ((u ^ (lane & 7)) << 4)) = make_uint4(pk[4 * u], pk[4 * u + 1], pk[4 * u + 2], pk[4 * u + 3]);
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        int cx = cx0 + c * 64, cy = cy0, cz = cz0, cu = cu0;
                        if (c_chunked) to_coords<FULL>(p.c, row0, n64, cx, cy, cz, cu);
                        tma_store_5d(mpc, buf, cx, cy, cz, cu, t.e * p.c.batched);
                        tma_store_commit();
                    }
                    ++epi_count;
                    return;
                }
                // a 64-column piece of a row is contiguous in every layout the GEMM accepts; rows past the tile's end
                // compute the address of its last row and store nothing (the row test only ever predicates a store:
                // the TMEM loads and waits around this code are warp-wide)
                const bool row_ok = m < t.m1;
                unsigned short* dst = p.C + c_offset<FULL>(p, min(m, t.m1 - 1), n64) + (int64_t)t.e * p.c_batch_stride;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (n64 + j * 8 < t.n1)              // the same for the whole warp; n1 - n0 is a multiple of 8
                        st_global_v4_if(dst + j * 8, make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]), row_ok);
            };
            // split-K: the fp32 partial sums of a piece, summed in fixed order by splitk_reduce_kernel
            auto store_partial = [&](const uint32_t (&r)[64], int c) {
                const int n64 = nb + c * 64;
                const bool row_ok = m < t.m1;
                float* wrow = p.ws + (((int64_t)t.e * p.splits + t.split) * p.M + min(m, t.m1 - 1)) * (int64_t)p.N;
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (n64 + j * 4 < t.n1)
                        st_global_v4_if(wrow + n64 + j * 4, make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]), row_ok);
            };
            // acc <- alpha * acc + beta * C for this lane's 64 columns (C read in its own layout, fp32 arithmetic)
            auto axpby_piece = [&](uint32_t (&r)[64], int c) {
                const int n64 = nb + c * 64;
                const bool row_ok = m < t.m1;
                const unsigned short* src = p.C + c_offset<FULL>(p, min(m, t.m1 - 1), n64) + (int64_t)t.e * p.c_batch_stride;
                const float alpha = p.alpha, beta = p.beta;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    uint4 cv = make_uint4(0u, 0u, 0u, 0u);
                    if (beta != 0.0f && n64 + j * 8 < t.n1) cv = ld_global_v4_if(src + j * 8, row_ok);
                    const uint32_t w[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {                       // bf16 -> fp32 is a shift
                        const float c0 = __uint_as_float(w[i] << 16), c1 = __uint_as_float(w[i] & 0xFFFF0000u);
                        r[j * 8 + 2 * i] = __float_as_uint(fmaf(alpha, __uint_as_float(r[j * 8 + 2 * i]), beta * c0));
                        r[j * 8 + 2 * i + 1] = __float_as_uint(fmaf(alpha, __uint_as_float(r[j * 8 + 2 * i + 1]), beta * c1));
                    }
                }
            };
            auto store_piece = [&](uint32_t (&r)[64], int c) {
                if (p.splits > 1) { store_partial(r, c); return; }
                if (FULL && p.axpby) axpby_piece(r, c);
                uint32_t pk[32];
                pack(r, pk);
                store_packed(pk, c);
            };
            // TMEM reads are software-pipelined: the load of piece c+1 is in flight while piece c is converted
            // and stored (two register sets, so the loop is unrolled by two).
            const int npieces = min((h == 0 ? SUBN : SUBN1) / 64, (t.n1 - nb + 63) / 64);      // warp-uniform
            uint32_t ra[64], rb[64];
            auto load_piece = [&](uint32_t (&r)[64], int c) {
                tmem_ld32(taddr + (uint32_t)(c * 64), *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
                tmem_ld32(taddr + (uint32_t)(c * 64 + 32), *reinterpret_cast<uint32_t(*)[32]>(&r[32]));
            };
            if (SWIGLU) {
                // piece c of accumulator 0 holds the gate values, piece c of accumulator 1 the up values of the same
                // 64 output columns: out = gate / (1 + exp(-gate)) * up, in fp32, then the usual bf16 store
#pragma unroll 1
                for (int c = hf; c < npieces; c += EW) {
                    load_piece(ra, c);
                    load_piece(rb, c + ACC_COLS / 64);
                    tmem_ld_wait();
                    tmem_regs_ready(ra);
                    tmem_regs_ready(rb);
                    uint32_t pk[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float g0 = __uint_as_float(ra[2 * i]), g1 = __uint_as_float(ra[2 * i + 1]);
                        const float u0 = __uint_as_float(rb[2 * i]), u1 = __uint_as_float(rb[2 * i + 1]);
                        const __nv_bfloat162 hh = __floats2bfloat162_rn(__fdividef(g0, 1.0f + __expf(-g0)) * u0,
                                                                        __fdividef(g1, 1.0f + __expf(-g1)) * u1);
                        pk[i] = *reinterpret_cast<const uint32_t*>(&hh);
                    }
                    store_packed(pk, c);
                }
            } else if (KS > 0) {
                // Cluster split: the KS CTAs of the cluster hold the partial sums of ONE tile, each over its part of K.  They
                // are exchanged in distributed shared memory -- no workspace, no second launch: of every 64-column piece,
                // CTA k of the cluster owns the 4-column groups [k JS, k JS + JS) (JS = 16 / KS); a warp instruction writes
                // one group of its 32 rows -- 512 contiguous bytes -- into the owner's copy of the operand ring, which all
                // MMAs are done with by then (first meeting of the cluster); after the second meeting every CTA sums its
                // column groups over the KS sources in the order of their k ranges (the same bits on every run), rounds
                // and stores them through C's layout.  (Tried and dropped: laying the sums out locally and sending one block
                // per destination with a bulk shared-to-shared copy that signals the destination's barrier -- 5 us slower
                // on the 256 x 768 x 2048 GEMM than these remote stores, which take ~80 cycles per 512-byte instruction.)
                constexpr int JS = 16 / (KS > 0 ? KS : 1), PP = BN / 64;
                cluster_sync();
                float* rbuf = reinterpret_cast<float*>(smem);                       // [source][quarter][piece][group in slice][lane] float4
#pragma unroll 1
                for (int c = 0; c < npieces; ++c) {
                    load_piece(ra, c);
                    tmem_ld_wait();
                    tmem_regs_ready(ra);
                    const uint32_t local = smem_u32(rbuf + ((((size_t)krank * 4 + quad) * PP + c) * JS * 32 + lane) * 4);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const uint32_t remote = map_to_cta(local + (uint32_t)(j % JS) * 512u, (uint32_t)(j / JS));   // owner j / JS, its slot j % JS
                        asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(remote), "r"(ra[4 * j]), "r"(ra[4 * j + 1]),
                                     "r"(ra[4 * j + 2]), "r"(ra[4 * j + 3]) : "memory");
                    }
                }
                cluster_sync();
                // (a tile lies inside one strip of C: the columns of a row follow each other from the tile's first column on)
                const int row = t.m0 + quad * 32 + lane;
                unsigned short* crow = p.C + c_offset<FULL>(p, min(row, t.m1 - 1), nb) + (int)krank * JS * 4;
#pragma unroll 1
                for (int c = 0; c < npieces; ++c)
#pragma unroll
                    for (int js = 0; js < JS; js += 2) {           // two 4-column groups = one 16-byte store
                        float4 a0 = make_float4(0.0f, 0.0f, 0.0f, 0.0f), a1 = a0;
#pragma unroll
                        for (int src = 0; src < KS; ++src) {
                            const float* g0 = rbuf + ((((size_t)src * 4 + quad) * PP + c) * JS * 32 + js * 32 + lane) * 4;
                            const float4 v0 = *reinterpret_cast<const float4*>(g0), v1 = *reinterpret_cast<const float4*>(g0 + 128);
                            a0.x += v0.x; a0.y += v0.y; a0.z += v0.z; a0.w += v0.w;
                            a1.x += v1.x; a1.y += v1.y; a1.z += v1.z; a1.w += v1.w;
                        }
                        const int col = nb + c * 64 + ((int)krank * JS + js) * 4;
                        if (p.axpby) {                             // C <- alpha * sum + beta * C (C read through its own layout)
                            const uint4 cv = ld_global_v4_if(crow + c * 64 + js * 4, p.beta != 0.0f && row < t.m1 && col < t.n1);
                            const float al = p.alpha, be = p.beta;
                            a0.x = fmaf(al, a0.x, be * __uint_as_float(cv.x << 16)); a0.y = fmaf(al, a0.y, be * __uint_as_float(cv.x & 0xFFFF0000u));
                            a0.z = fmaf(al, a0.z, be * __uint_as_float(cv.y << 16)); a0.w = fmaf(al, a0.w, be * __uint_as_float(cv.y & 0xFFFF0000u));
                            a1.x = fmaf(al, a1.x, be * __uint_as_float(cv.z << 16)); a1.y = fmaf(al, a1.y, be * __uint_as_float(cv.z & 0xFFFF0000u));
                            a1.z = fmaf(al, a1.z, be * __uint_as_float(cv.w << 16)); a1.w = fmaf(al, a1.w, be * __uint_as_float(cv.w & 0xFFFF0000u));
                        }
                        const __nv_bfloat162 h0 = __floats2bfloat162_rn(a0.x, a0.y), h1 = __floats2bfloat162_rn(a0.z, a0.w);
                        const __nv_bfloat162 h2 = __floats2bfloat162_rn(a1.x, a1.y), h3 = __floats2bfloat162_rn(a1.z, a1.w);
                        uint4 o;
                        o.x = *reinterpret_cast<const uint32_t*>(&h0); o.y = *reinterpret_cast<const uint32_t*>(&h1);
                        o.z = *reinterpret_cast<const uint32_t*>(&h2); o.w = *reinterpret_cast<const uint32_t*>(&h3);
                        st_global_v4_if(crow + c * 64 + js * 4, o, row < t.m1 && col < t.n1);
                    }
            } else if (bal && t.part != 0) {
                // Balanced split, a tile shared by t.nshare units.  A unit's slot of the workspace holds one CTA's 128 x BN
                // partial sums as [epilogue warp][64-column piece][16][lane] float4 -- the registers of a piece exactly as
                // tcgen05.ld hands them out, so a warp reads and writes 512 contiguous bytes per instruction; the flags of all
                // CTAs follow the slots.
                // A unit's share can end in one tile and go on in the next: a CTA has two slots (and two sets of flags), the
                // first for a share that starts inside a tile, the second for the share that starts a tile (k = 0).
                const size_t slot_floats = (size_t)BM * BN, quad_off = (size_t)quad * 32 * BN;
                constexpr int PPS = SUBN / 64;                     // pieces per sub-tile
                const size_t my_slot = (size_t)blockIdx.x * 2 + (t.mine == 0 ? 1 : 0);
                // (1) this sub-tile's partial sums -> own slot; the accumulator goes back to the tensor cores at once
#pragma unroll 1
                for (int c = 0; c < npieces; ++c) {
                    load_piece(ra, c);
                    tmem_ld_wait();
                    tmem_regs_ready(ra);
                    float* dst = p.ws + my_slot * slot_floats + quad_off + (size_t)(h * PPS + c) * (32 * 64) + (size_t)lane * 4;
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        *reinterpret_cast<uint4*>(dst + j * 128) = make_uint4(ra[4 * j], ra[4 * j + 1], ra[4 * j + 2], ra[4 * j + 3]);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (CTAS == 2) mbar_arrive_cluster(tmem_empty0 + (uint32_t)acc * 8u);
                    else mbar_arrive(&tmem_empty[acc]);
                }
                released = true;
                if (h == NSUB - 1) {
                    // (2) mark this warp's rows of the share as written
                    __threadfence();
                    __syncwarp();
                    if (lane == 0) asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p.bal_flags + my_slot * 4 + quad), "l"(p.bal_mark) : "memory");
                    // (3) the reduction of a shared tile waits for the other sharers; if this unit's next piece of work is
                    // another share, that one is written first -- its sharers wait for it in turn, and a unit that reduced
                    // before writing would make them queue up one behind the other across the whole group
                    pend[npend++] = t;
                    TileCoord nx;
                    const bool more = sched.template get<RAG, FULL>(it + 1, nx);
                    if (!(more && nx.part != 0)) {
                        for (int q = 0; q < npend && alive; ++q) {
                            t = pend[q];
                            m = t.m0 + (int)rank * BM + quad * 32 + lane;
                            row0 = t.m0 + (int)rank * BM + quad * 32;
                            rows_full = row0 + 32 <= t.m1;
                            const int cta0 = (int)blockIdx.x - t.mine * CTAS;       // the first sharer's CTA of this rank
                            bool seen = true;                                       // bounded wait for the same rows of the other sharers
                            const uint64_t t0 = global_timer_ns();
                            for (int o = 0; seen && o < t.nshare; ++o) {
                                if (o == t.mine) continue;
                                const unsigned long long* f = p.bal_flags + ((size_t)(cta0 + o * CTAS) * 2 + (o == 0 ? 1 : 0)) * 4 + quad;
                                while (ld_acquire_u64(f) != p.bal_mark)
                                    if (global_timer_ns() - t0 > kWaitLimitNs) { seen = false; break; }
                            }
                            seen = __all_sync(0xffffffffu, seen);
                            if (!seen) { if (lane == 0) atomicExch(&g_gemm_status, 7); alive = false; break; }
                            // every nshare-th piece of the tile is this unit's: sum the sharers' partial sums in the order of
                            // their k ranges (the same bits on every run) and store the piece as usual
#pragma unroll 1
                            for (int hh = 0; hh < NSUB; ++hh) {
                                nb = t.n0 + hh * SUBN;
                                to_coords<FULL>(p.c, row0, nb, cx0, cy0, cz0, cu0);
                                const int np = min(PPS, (t.n1 - nb + 63) / 64);
#pragma unroll 1
                                for (int c = 0; c < np; ++c) {
                                    const int pc = hh * PPS + c;
                                    if (pc % t.nshare != t.mine) continue;
                                    const size_t piece_off = quad_off + (size_t)pc * (32 * 64) + (size_t)lane * 4;
#pragma unroll 1
                                    for (int o = 0; o < t.nshare; ++o) {
                                        const float* src = p.ws + ((size_t)(cta0 + o * CTAS) * 2 + (o == 0 ? 1 : 0)) * slot_floats + piece_off;
#pragma unroll
                                        for (int j = 0; j < 16; ++j) {             // sixteen loads in flight, then the sums
                                            const uint4 v = __ldcg(reinterpret_cast<const uint4*>(src + j * 128));
                                            rb[4 * j] = v.x; rb[4 * j + 1] = v.y; rb[4 * j + 2] = v.z; rb[4 * j + 3] = v.w;
                                        }
                                        if (o == 0) {
#pragma unroll
                                            for (int i = 0; i < 64; ++i) ra[i] = rb[i];
                                        } else {
#pragma unroll
                                            for (int i = 0; i < 64; ++i) ra[i] = __float_as_uint(__uint_as_float(ra[i]) + __uint_as_float(rb[i]));
                                        }
                                    }
                                    store_piece(ra, c);
                                }
                            }
                        }
                        npend = 0;
                        if (!alive) break;
                    }
                }
            } else if (EW > 1) {
#pragma unroll 1
                for (int c = hf; c < npieces; c += EW) {
                    load_piece(ra, c);
                    tmem_ld_wait();
                    tmem_regs_ready(ra);
                    store_piece(ra, c);
                }
            } else {
            if (npieces > 0) load_piece(ra, 0);
#pragma unroll 1
            for (int c = 0; c < npieces; c += 2) {
                tmem_ld_wait();
                tmem_regs_ready(ra);
                if (c + 1 < npieces) load_piece(rb, c + 1);
                store_piece(ra, c);
                if (c + 1 < npieces) {
                    tmem_ld_wait();
                    tmem_regs_ready(rb);
                    if (c + 2 < npieces) load_piece(ra, c + 2);
                    store_piece(rb, c + 1);
                }
            }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0 && !released) {
                if (CTAS == 2) mbar_arrive_cluster(tmem_empty0 + (uint32_t)acc * 8u);
                else mbar_arrive(&tmem_empty[acc]);
                if (SWIGLU) {                            // both accumulators of the tile have been read
                    if (CTAS == 2) mbar_arrive_cluster(tmem_empty0 + 8u);
                    else mbar_arrive(&tmem_empty[1]);
                }
            }
          }
        }
        // every tile store has read its shared-memory source; the writes themselves are complete, like any other
        // store of the kernel, when the kernel is
        if (lane == 0) tma_store_wait_read<0>();
    }

    tc_fence_before();
    __syncthreads();
    if (CTAS == 2) cluster_sync();                   // neither CTA frees TMEM or exits while the other may still use it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<CTAS>(tmem_base, kTmemCols);
    }
}

// Split-K epilogue: C = bf16( ws[0] + ws[1] + ... + ws[splits-1] ), the sum taken in that fixed order so
// the result is the same on every run.  One thread per 8 consecutive columns of a row.
__global__ void __launch_bounds__(256) splitk_reduce_kernel(const GemmParams p) {
    const int64_t n8 = p.N / 8, per_problem = (int64_t)p.M * n8, total = per_problem * p.batch;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t e = i / per_problem, r = i - e * per_problem;
        const int64_t m = r / n8, n = (r - m * n8) * 8;
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = 0.0f;
        for (int sp = 0; sp < p.splits; ++sp) {
            const float4* src = reinterpret_cast<const float4*>(p.ws + ((e * p.splits + sp) * p.M + m) * (int64_t)p.N + n);
            const float4 x = src[0], y = src[1];
            acc[0] += x.x; acc[1] += x.y; acc[2] += x.z; acc[3] += x.w;
            acc[4] += y.x; acc[5] += y.y; acc[6] += y.z; acc[7] += y.w;
        }
        const int64_t off = c_offset(p, m, n) + e * p.c_batch_stride;
        if (p.axpby) {
            uint4 cv = make_uint4(0u, 0u, 0u, 0u);
            if (p.beta != 0.0f) cv = *reinterpret_cast<const uint4*>(p.C + off);
            const uint32_t w[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                acc[2 * i] = fmaf(p.alpha, acc[2 * i], p.beta * __uint_as_float(w[i] << 16));
                acc[2 * i + 1] = fmaf(p.alpha, acc[2 * i + 1], p.beta * __uint_as_float(w[i] & 0xFFFF0000u));
            }
        }
        uint4 v;
        __nv_bfloat162 h;
        h = __floats2bfloat162_rn(acc[0], acc[1]); v.x = *reinterpret_cast<uint32_t*>(&h);
        h = __floats2bfloat162_rn(acc[2], acc[3]); v.y = *reinterpret_cast<uint32_t*>(&h);
        h = __floats2bfloat162_rn(acc[4], acc[5]); v.z = *reinterpret_cast<uint32_t*>(&h);
        h = __floats2bfloat162_rn(acc[6], acc[7]); v.w = *reinterpret_cast<uint32_t*>(&h);
        *reinterpret_cast<uint4*>(p.C + off) = v;
    }
}

}  // namespace ccl

#endif  // CCL_GEMM_KERNEL_CUH_
