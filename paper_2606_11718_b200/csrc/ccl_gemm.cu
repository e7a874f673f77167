// ccl_gemm: bf16 GEMM (fp32 accumulate, bf16 RNE output) whose A / B / C live in row-major or
// Chiplet-Contiguous Layout (Sec. 2.2 execution model; Sec. 3.3: only the address map changes).
//
// Design (sm_100a):
//   * CCL is folded into TMA tensor maps {strip-local contiguous extent, rows, strip, 1}
//     -- the view (K, G, N/G) with strides (w, K*w, 1) of Sec. 3.3 -- so the address
//     translation costs nothing per access and a partial last tile of a strip is handled by
//     TMA zero fill.  The page-interleaved form of CCL uses the fourth dimension: the chunk
//     index (chunks of whole rows) or the chunk within a row (rows of whole chunks).
//   * Persistent, warp-specialised CTAs: warp 0 = TMA producer, warp 1 = tcgen05.mma issuer
//     (the warp runs the issue loop on warp-uniform values, one elected lane issues) and TMEM
//     owner, warps 2-5 = epilogue (TMEM -> registers -> bf16 -> global, addressing C through
//     its own layout).
//   * Two flavours of one kernel template:
//       CTAS = 2: a cluster of two CTAs (one SM pair) computes a 256 x BN tile with
//                 tcgen05.mma.cta_group::2; each CTA stages its own 128 rows of A and its own
//                 half of the B columns, which halves the operand bytes an SM pulls per flop;
//       CTAS = 1: one CTA per 128 x BN tile, for shapes whose M extent does not fill a pair.
//   * SWIZZLE_128B shared-memory tiles, a ring of smem stages, two TMEM accumulators so the
//     epilogue of tile i overlaps the main loop of tile i+1.
//   * Chiplet-grouped raster (Sec. 3.1): the CTAs are cut into P groups and group g walks only
//     the output tiles of strip g, i.e. it streams one contiguous region of B and C.
//   * Every mbarrier wait is bounded; on expiry the kernel records a code in g_gemm_status,
//     all roles leave their loops, TMEM is released and the kernel returns.
//
// Files: ccl_gemm_kernel.cuh (the kernel and its device helpers), ccl_gemm_plan.cuh (planning: checks, cost model, tensor
// maps), this file (launch, the cache of prepared calls, the C entry points).
#include "ccl_gemm_kernel.cuh"
#include "ccl_gemm_plan.cuh"

namespace ccl {

template <int BN, int CTAS, bool SWIGLU = false, int RAG = 0, bool FULL = true, int KS = 0>
static ccl_status configure(uint32_t smem_bytes) {
    static uint32_t configured_for = 0;
    if (configured_for < smem_bytes) {
        CCL_CUDA_TRY(cudaFuncSetAttribute(ccl_gemm_kernel<BN, CTAS, SWIGLU, RAG, FULL, KS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes));
        configured_for = smem_bytes;
    }
    return CCL_OK;
}

template <int BN, int CTAS, bool SWIGLU = false, int RAG = 0, bool FULL = true, int KS = 0>
static ccl_status launch(const GemmPlan& plan, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, cudaStream_t st) {
    ccl_status s = configure<BN, CTAS, SWIGLU, RAG, FULL, KS>(plan.smem_bytes);
    if (s) return s;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.grid, 1, 1);
    cfg.blockDim = dim3(kGemmThreads, 1, 1);
    cfg.dynamicSmemBytes = plan.smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = KS ? KS : CTAS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // Programmatic dependent launch (CCL_GEMM_PDL=0 turns it off): this kernel's CTAs may be placed, and run their set-up
    // (parameters, barriers, TMEM, tensor-map prefetch), while the previous kernel in the stream drains; they touch
    // global memory only after griddepcontrol.wait, i.e. after that kernel has completed and flushed.
    static const bool pdl = []() { const char* f = std::getenv("CCL_GEMM_PDL"); return !f || atoi(f) != 0; }();
    if (pdl) {
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.numAttrs = 2;
    }
    CCL_CUDA_TRY(cudaLaunchKernelEx(&cfg, ccl_gemm_kernel<BN, CTAS, SWIGLU, RAG, FULL, KS>, ma, mb, mc, plan.ma2, plan.mb2, plan.mc2, plan.p));
    count_launch();
    return CCL_OK;
}

// CTA pairs of the 2-CTA kernel that can be resident at once (0 if clusters cannot be launched)
static int resident_pairs() {
    static int pairs = -1;
    if (pairs >= 0) return pairs;
    uint32_t smem = kSmemBudget + kEpiBytes + 2048;
    if (configure<256, 2>(smem) != CCL_OK) { clear_error(); return pairs = 0; }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2, 1, 1); cfg.blockDim = dim3(kGemmThreads, 1, 1); cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, ccl_gemm_kernel<256, 2>, &cfg) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
    return pairs = n;
}

// Clusters of `ks` CTAs of the cluster-split kernel that can be resident at once (a tile per cluster); the figures of a
// B200 (16 clusters of 8, 32 of 4, 64 of 2: clusters do not span GPCs) when no device can be asked.
template <int KS>
static int query_clusters() {
    uint32_t smem = kSmemBudget + kEpiBytes + 2048;
    if (configure<256, 1, false, 0, false, KS>(smem) != CCL_OK) { clear_error(); return 0; }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(KS, 1, 1); cfg.blockDim = dim3(kGemmThreads, 1, 1); cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = KS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, ccl_gemm_kernel<256, 1, false, 0, false, KS>, &cfg) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
    return n;
}
static int resident_clusters(int ks, bool have_device) {
    static int cached[9] = {-1, -1, -1, -1, -1, -1, -1, -1, -1};
    if (!have_device) return ks == 2 ? 64 : (ks == 4 ? 32 : 16);
    if (cached[ks] < 0) cached[ks] = ks == 2 ? query_clusters<2>() : (ks == 4 ? query_clusters<4>() : query_clusters<8>());
    return cached[ks];
}

ccl_status repack_status_take(int* code);   // ccl_repack.cu
ccl_status repack_selftest_launch(const void* src_dev, uint64_t limit_ns, cudaStream_t st);   // ccl_repack.cu

// Self-test of the GEMM's expiry path (ccl_selftest_wait_timeout, which = 0): one CTA allocates TMEM like the GEMM,
// one thread waits -- bounded -- on an mbarrier nobody ever arrives at, records code 6 in the status word when the wait
// gives up, and the CTA leaves the way the GEMM does: block-wide sync, TMEM released.
__global__ void __launch_bounds__(64) wait_selftest_kernel(uint64_t limit_ns) {
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) { mbar_init(&bar, 1); fence_barrier_init(); }
    if (warp == 1) tmem_alloc<1>(&tmem_slot, 32);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    if (threadIdx.x == 0 && !mbar_wait_bounded(&bar, 0u, limit_ns)) atomicExch(&g_gemm_status, 6);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc_fence_after(); tmem_dealloc<1>(tmem_base, 32); }
}

}  // namespace ccl

using namespace ccl;

// ---- host-side cache of prepared calls (plan + encoded tensor maps) --------------------------------------
struct PreparedKey {
    int64_t f[40];          // every field of the descriptor, the batch, the three pointers, the ragged-batch arguments, the workspace at hand
    int dev;
    int mode;               // 0 plain, 1 gated activation
    float alpha, beta;
    char env[60];
};
struct Prepared {
    PreparedKey key;
    GemmPlan plan;
    CUtensorMap ma, mb, mc;
    int sms;
    bool valid = false;
};
constexpr int kPreparedSlots = 16;
static Prepared g_prepared[kPreparedSlots];
static int g_prepared_next = 0;
static std::mutex g_prepared_mutex;

static void put_mat(const ccl_mat& m, int64_t* f) {
    f[0] = m.rows; f[1] = m.cols; f[2] = m.elem_bytes; f[3] = m.P; f[4] = m.part; f[5] = m.layout; f[6] = m.strip_align_bytes;
}
static void make_key(const ccl_gemm_desc* d, const int64_t* batch4, const void* A, const void* B, const void* C, PreparedKey* k) {
    std::memset(k, 0, sizeof(*k));
    for (int i = 0; i < 4; ++i) k->f[32 + i] = batch4[i];          // batch, strides of A, B, C
    k->f[0] = d->M; k->f[1] = d->N; k->f[2] = d->K;
    put_mat(d->A, k->f + 3); put_mat(d->B, k->f + 10); put_mat(d->C, k->f + 17);
    k->f[24] = d->a_trans; k->f[25] = d->b_trans; k->f[26] = d->out_part; k->f[27] = d->P;
    k->f[28] = d->grouped_raster + ((int64_t)(d->out_part == CCL_PART_2D ? d->part_m : 0) << 8);
    k->f[29] = (int64_t)reinterpret_cast<uintptr_t>(A); k->f[30] = (int64_t)reinterpret_cast<uintptr_t>(B);
    k->f[31] = (int64_t)reinterpret_cast<uintptr_t>(C);
    k->dev = -1;
    (void)cudaGetDevice(&k->dev);
    size_t pos = 0;
    for (const char* name : {"CCL_GEMM_CTAS", "CCL_GEMM_BN", "CCL_GEMM_SPLITK", "CCL_GEMM_RAGGED_DENSE", "CCL_GEMM_BALANCED", "CCL_GEMM_CLUSTERK"}) {
        const char* v = std::getenv(name);
        for (const char* c = v ? v : ""; *c && pos + 2 < sizeof(k->env); ++c) k->env[pos++] = *c;
        if (pos + 1 < sizeof(k->env)) k->env[pos++] = ';';
    }
}

// SM count and resident CTA pairs of the current device; the figures of a B200 when no device is usable
// (the planner then still validates and sizes the workspace the same way a B200 would).
static bool device_units(int* sms, int* pairs) {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) {
        *sms = n; *pairs = resident_pairs();
        return true;
    }
    (void)cudaGetLastError();
    *sms = 148; *pairs = 74;
    return false;
}

constexpr int64_t kMaxBatch = 65536;

static ccl_status workspace_impl(const ccl_gemm_desc* d, int64_t batch, size_t* bytes) {
    if (batch < 1 || batch > kMaxBatch) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm: batch must be in [1, %lld]", (long long)kMaxBatch);
    GemmPlan plan;
    ccl_status s = make_plan(d, batch, false, nullptr, nullptr, nullptr, 148, 74, &plan);     // validation without any CUDA call
    if (s) return s;
    if (!bytes) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm_workspace: NULL output");
    int sms, pairs;
    const bool have_device = device_units(&sms, &pairs);
    if ((s = make_plan(d, batch, false, nullptr, nullptr, nullptr, sms, pairs, &plan, 0, false, ~(size_t)0, have_device))) return s;
    *bytes = plan.ws_bytes;
    return CCL_OK;
}

extern "C" ccl_status ccl_gemm_workspace(const ccl_gemm_desc* d, size_t* bytes) { return workspace_impl(d, 1, bytes); }
extern "C" ccl_status ccl_gemm_batched_workspace(const ccl_gemm_desc* d, int32_t batch, size_t* bytes) { return workspace_impl(d, batch, bytes); }

// Scratch for the split-K partial sums, part of the library image: every GPU that loads the library
// holds these bytes until the process ends.  Only device code may use the name as an address; on the
// host the name is merely a handle that cudaGetSymbolAddress turns into the device pointer.
static __device__ __align__(256) unsigned char g_static_ws[CCL_GEMM_STATIC_WS_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_ws_mutex;
void* g_static_ws_addr[kMaxDevices] = {};

// Device address of g_static_ws on the current device, looked up once per device.
ccl_status static_ws_address(void** out) {
    int dev = -1;
    CCL_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return ccl::fail(CCL_ERR_UNSUPPORTED, "ccl_gemm_static_ws: device ordinal %d is beyond the %d this library tracks", dev, kMaxDevices);
    std::lock_guard<std::mutex> lock(g_static_ws_mutex);
    if (!g_static_ws_addr[dev]) {
        void* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_ws);
        if (e != cudaSuccess || !ptr)
            return ccl::fail(CCL_ERR_CUDA, "ccl_gemm_static_ws: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
        g_static_ws_addr[dev] = ptr;
    }
    *out = g_static_ws_addr[dev];
    return CCL_OK;
}
}  // namespace

// strides[X]: bytes between the buffers of operand X (A, B, C) of consecutive problems; 0 = shared (A and B only)
// m_offs / cap: ragged batch (ccl_gemm_grouped), else nullptr / 0
static ccl_status gemm_impl(const ccl_gemm_desc* d, int64_t batch, bool swiglu, const int64_t* strides, const void* A_dev, const void* B_dev, void* C_dev,
                            void* ws_dev, size_t ws_bytes, void* cuda_stream, float alpha = 1.0f, float beta = 0.0f, const int32_t* m_offs = nullptr,
                            int64_t cap = 0, const int32_t* k_offs = nullptr, bool static_ws = false) {
    if (!A_dev || !B_dev || !C_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm: NULL operand");
    if (!d) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm: NULL descriptor");
    if (batch < 1 || batch > kMaxBatch) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm: batch must be in [1, %lld]", (long long)kMaxBatch);
    const int64_t batch4[4] = {batch, batch > 1 ? strides[0] : 0, batch > 1 ? strides[1] : 0, batch > 1 ? strides[2] : 0};
    // Repeated calls with the same descriptor and buffers (the normal case in a training / serving loop)
    // reuse the plan and the two encoded tensor maps: a host-side cache only, nothing is kept on the device.
    PreparedKey key;
    make_key(d, batch4, A_dev, B_dev, C_dev, &key);
    key.mode = (swiglu ? 1 : 0) | (static_ws ? 2 : 0); key.alpha = alpha; key.beta = beta;
    key.f[36] = (int64_t)reinterpret_cast<uintptr_t>(m_offs) ^ ((int64_t)reinterpret_cast<uintptr_t>(k_offs) << 1); key.f[37] = cap + (k_offs ? (INT64_C(1) << 62) : 0);
    // The balanced split is optional: it is planned only when the workspace at hand holds its partial sums (the caller's
    // ws_bytes; the scratch array for ccl_gemm_static_ws).  A caller that passes none gets whole-tile plans, as before.
    const size_t max_ws = static_ws ? (size_t)CCL_GEMM_STATIC_WS_BYTES : (ws_dev ? ws_bytes : 0);
    key.f[38] = (int64_t)max_ws;
    Prepared prep;
    bool hit = false;
    {
        std::lock_guard<std::mutex> lock(g_prepared_mutex);
        for (int i = 0; i < kPreparedSlots; ++i)
            if (g_prepared[i].valid && std::memcmp(&g_prepared[i].key, &key, sizeof(key)) == 0) { prep = g_prepared[i]; hit = true; break; }
    }
    ccl_status s;
    if (!hit) {
        GemmPlan& plan = prep.plan;
        s = make_plan(d, batch, swiglu, A_dev, B_dev, C_dev, 148, 74, &plan, cap, k_offs != nullptr, max_ws);     // validation first: no CUDA call on bad input
        if (s) return s;
        if (batch > 1) {
            const MatView* views[3] = {&plan.va, &plan.vb, &plan.vc};
            const char* names[3] = {"A", "B", "C"};
            for (int X = 0; X < 3; ++X) {
                const int64_t st = batch4[1 + X], need = buffer_elems(*views[X]) * 2;
                if (st == 0 && (X < 2 || m_offs)) continue;         // an operand every problem shares (or, ragged, one concatenated C)
                if (st < need) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm_batched: stride of %s (%lld bytes) is smaller than its buffer (%lld bytes)", names[X], (long long)st, (long long)need);
                if (st % 16) return fail(CCL_ERR_ALIGN, "ccl_gemm_batched: stride of %s is not a multiple of 16 bytes", names[X]);
                if (st >= (INT64_C(1) << 40)) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm_batched: stride of %s too large for a tensor map", names[X]);
            }
        }
        int dev;
        CCL_CUDA_TRY(cudaGetDevice(&dev));
        CCL_CUDA_TRY(cudaDeviceGetAttribute(&prep.sms, cudaDevAttrMultiProcessorCount, dev));
        if (dev != key.dev) {
            make_key(d, batch4, A_dev, B_dev, C_dev, &key);
            key.mode = (swiglu ? 1 : 0) | (static_ws ? 2 : 0); key.alpha = alpha; key.beta = beta; key.f[38] = (int64_t)max_ws;
            key.f[36] = (int64_t)reinterpret_cast<uintptr_t>(m_offs) ^ ((int64_t)reinterpret_cast<uintptr_t>(k_offs) << 1); key.f[37] = cap + (k_offs ? (INT64_C(1) << 62) : 0);
        }
        if ((s = make_plan(d, batch, swiglu, A_dev, B_dev, C_dev, prep.sms, resident_pairs(), &plan, cap, k_offs != nullptr, max_ws, true))) return s;
        plan.p.C = static_cast<uint16_t*>(C_dev);
        plan.p.a.batched = batch4[1] != 0; plan.p.b.batched = batch4[2] != 0; plan.p.c.batched = m_offs ? 0 : 1;
        plan.p.m_offs = m_offs;
        plan.p.k_offs = k_offs;
        plan.p.c_batch_stride = batch4[3] / 2;
        plan.p.alpha = alpha; plan.p.beta = beta; plan.p.axpby = (alpha != 1.0f || beta != 0.0f) ? 1 : 0;
        {
            const GemmParams& q = plan.p;
            const bool ks = (q.a_mn ? q.a.split == 1 : q.a.split == 2) || (q.b_mn ? q.b.split == 1 : q.b.split == 2);
            plan.lean = q.group_dim != 2 && !q.axpby && batch == 1 && !q.a.il_mode && !q.b.il_mode && !q.c.il_mode && !ks && !m_offs && !k_offs && !swiglu &&
                        !q.a.rag && !q.b.rag && !q.c.rag;
        }
        const uint32_t bnh = plan.bn == 384 ? 64u : (uint32_t)(plan.subn / plan.ctas);   // B rows of one K-major box
        if (!plan.p.a_mn) s = operand_tmap(&prep.ma, plan.va, A_dev, BK, (uint32_t)plan.a_box_rows, batch, batch4[1]); else s = operand_tmap(&prep.ma, plan.va, A_dev, 64, BK, batch, batch4[1]);
        if (s) return s;
        if (!plan.p.b_mn) s = operand_tmap(&prep.mb, plan.vb, B_dev, BK, bnh, batch, batch4[2]); else s = operand_tmap(&prep.mb, plan.vb, B_dev, 64, BK, batch, batch4[2]);
        if (s) return s;
        if ((s = operand_tmap(&prep.mc, plan.vc, C_dev, 64, 32, batch, batch4[3]))) return s;   // C: 64-column x 32-row store boxes
        // the last strips of operands whose strips are not all alike (else copies)
        plan.ma2 = prep.ma; plan.mb2 = prep.mb; plan.mc2 = prep.mc;
        if (ragged(plan.va) && (s = plan.p.a_mn ? operand_tmap(&plan.ma2, plan.va, A_dev, 64, BK, batch, batch4[1], true)
                                              : operand_tmap(&plan.ma2, plan.va, A_dev, BK, (uint32_t)plan.a_box_rows, batch, batch4[1], true))) return s;
        if (ragged(plan.vb) && (s = plan.p.b_mn ? operand_tmap(&plan.mb2, plan.vb, B_dev, 64, BK, batch, batch4[2], true)
                                              : operand_tmap(&plan.mb2, plan.vb, B_dev, BK, bnh, batch, batch4[2], true))) return s;
        if (ragged(plan.vc) && (s = operand_tmap(&plan.mc2, plan.vc, C_dev, 64, 32, batch, batch4[3], true))) return s;
        prep.key = key; prep.valid = true;
        std::lock_guard<std::mutex> lock(g_prepared_mutex);
        g_prepared[g_prepared_next] = prep;
        g_prepared_next = (g_prepared_next + 1) % kPreparedSlots;
    }
    GemmPlan& plan = prep.plan;
    const CUtensorMap &ma = prep.ma, &mb = prep.mb, &mc = prep.mc;
    const int sms = prep.sms;
    if (static_ws) {                                     // ccl_gemm_static_ws: the scratch compiled into the library image
        if (plan.ws_bytes > (size_t)CCL_GEMM_STATIC_WS_BYTES)
            return fail(CCL_ERR_WORKSPACE, "ccl_gemm_static_ws: this problem needs %zu bytes of split-K workspace, the built-in scratch holds %u; "
                        "use ccl_gemm with a caller-provided workspace", plan.ws_bytes, (unsigned)CCL_GEMM_STATIC_WS_BYTES);
        ws_dev = nullptr; ws_bytes = 0;
        if (plan.ws_bytes) {
            if ((s = static_ws_address(&ws_dev))) return s;
            ws_bytes = (size_t)CCL_GEMM_STATIC_WS_BYTES;
        }
    }
    if (plan.ws_bytes) {
        if (!ws_dev || ws_bytes < plan.ws_bytes)
            return fail(CCL_ERR_WORKSPACE, "ccl_gemm: this problem is split along K and needs %zu bytes of workspace (got %zu)", plan.ws_bytes, ws_dev ? ws_bytes : (size_t)0);
        if (reinterpret_cast<uintptr_t>(ws_dev) & 15) return fail(CCL_ERR_ALIGN, "ccl_gemm: workspace is not 16-byte aligned");
    }
    plan.p.ws = static_cast<float*>(ws_dev);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    if (plan.p.bal) {                                    // flags behind the partial sums, cleared in front of the launch
        plan.p.bal_flags = reinterpret_cast<unsigned long long*>(static_cast<char*>(ws_dev) + (size_t)plan.grid * 2 * ((size_t)BM * plan.bn * 4));
        plan.p.bal_mark = 1ull;
        CCL_CUDA_TRY(cudaMemsetAsync(plan.p.bal_flags, 0, (size_t)plan.grid * 2 * 32, st));
    }
    // Soft wave barrier for problems of three or more full rounds of tiles (CCL_GEMM_WAVESYNC=0 turns it off, =n syncs
    // every n-th round): without it the CTAs that share an A panel or B
    // columns drift apart by more than the L2 holds and fetch the same lines from DRAM 2-3 times.
    plan.p.wave_ctr = nullptr;
    {
        static const int wave_sync = []() { const char* f = std::getenv("CCL_GEMM_WAVESYNC"); return f ? atoi(f) : 1; }();
        plan.p.wave_period = wave_sync > 0 ? wave_sync : 1; plan.p.wave_wait_ns = 20000;        // one wait gives up after 20 us
        // (long tiles only: with K below 4096, or a batch of small problems, the CTAs share little and the waits only cost --
        // measured -9 % on 128 batched expert GEMMs and on a 16384 x 1536 x 2048 fused gate/up GEMM)
        const bool any_rag = plan.p.a.rag || plan.p.b.rag || plan.p.c.rag;      // (CTAs that skip the empty places of a short last strip would miss the meeting)
        if (wave_sync > 0 && plan.p.sch_rounds >= 3 && plan.p.kb_per_split >= 64 && batch == 1 && !m_offs && !k_offs && !any_rag) {
            // One of kWaveSlots counters in the library image, handed out round-robin: a launch recorded into a CUDA graph
            // keeps its slot for good while eager calls rotate through all of them, so two GEMMs that overlap on the GPU
            // can land on one counter -- the barrier is soft (a wait just ends early or runs into its 20 us bound), results
            // never depend on it.  A device ordinal beyond the table runs without the barrier.
            static std::atomic<unsigned int> next{0};
            static std::mutex base_mutex;
            static unsigned int* base[64] = {};                  // address of the counters, per device
            int dev = 0;
            CCL_CUDA_TRY(cudaGetDevice(&dev));
            unsigned int* ctr0 = nullptr;
            if (dev >= 0 && dev < 64) {
                std::lock_guard<std::mutex> lock(base_mutex);
                if (!base[dev]) CCL_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&base[dev]), g_wave_ctr));
                ctr0 = base[dev];
            }
            if (ctr0) {
                plan.p.wave_ctr = ctr0 + next.fetch_add(1) % kWaveSlots;
                CCL_CUDA_TRY(cudaMemsetAsync(plan.p.wave_ctr, 0, sizeof(unsigned int), st));
            }
        }
    }
    if (k_offs) {                                        // ragged K: one CTA per tile (make_plan)
        if (plan.bn == 256) s = launch<256, 1, false, 2>(plan, ma, mb, mc, st);
        else if (plan.bn == 192) s = launch<192, 1, false, 2>(plan, ma, mb, mc, st);
        else s = launch<128, 1, false, 2>(plan, ma, mb, mc, st);
    } else if (m_offs) {                                 // ragged M
        if (swiglu) s = launch<512, 2, true, 1>(plan, ma, mb, mc, st);
        else if (plan.ctas == 2) {
            if (plan.bn == 512) s = launch<512, 2, false, 1>(plan, ma, mb, mc, st);
            else if (plan.bn == 192) s = launch<192, 2, false, 1>(plan, ma, mb, mc, st);
            else s = plan.bn == 256 ? launch<256, 2, false, 1>(plan, ma, mb, mc, st) : launch<128, 2, false, 1>(plan, ma, mb, mc, st);
        } else if (plan.bn == 256) s = launch<256, 1, false, 1>(plan, ma, mb, mc, st);
        else if (plan.bn == 192) s = launch<192, 1, false, 1>(plan, ma, mb, mc, st);
        else s = launch<128, 1, false, 1>(plan, ma, mb, mc, st);
    } else if (swiglu) s = launch<512, 2, true>(plan, ma, mb, mc, st);
    else if (plan.ks) {                                  // cluster split along K (plain calls only)
        const int key = plan.bn * 10 + plan.ks;
        if (key == 2562) s = launch<256, 1, false, 0, false, 2>(plan, ma, mb, mc, st);
        else if (key == 2564) s = launch<256, 1, false, 0, false, 4>(plan, ma, mb, mc, st);
        else if (key == 2568) s = launch<256, 1, false, 0, false, 8>(plan, ma, mb, mc, st);
        else if (key == 1922) s = launch<192, 1, false, 0, false, 2>(plan, ma, mb, mc, st);
        else if (key == 1924) s = launch<192, 1, false, 0, false, 4>(plan, ma, mb, mc, st);
        else if (key == 1928) s = launch<192, 1, false, 0, false, 8>(plan, ma, mb, mc, st);
        else if (key == 1282) s = launch<128, 1, false, 0, false, 2>(plan, ma, mb, mc, st);
        else if (key == 1284) s = launch<128, 1, false, 0, false, 4>(plan, ma, mb, mc, st);
        else s = launch<128, 1, false, 0, false, 8>(plan, ma, mb, mc, st);
    } else if (plan.lean) {                                // nothing optional in use: the instantiation without those branches
        if (plan.ctas == 2) {
            if (plan.bn == 512) s = launch<512, 2, false, 0, false>(plan, ma, mb, mc, st);
            else if (plan.bn == 384) s = launch<384, 2, false, 0, false>(plan, ma, mb, mc, st);
            else if (plan.bn == 192) s = launch<192, 2, false, 0, false>(plan, ma, mb, mc, st);
            else s = plan.bn == 256 ? launch<256, 2, false, 0, false>(plan, ma, mb, mc, st) : launch<128, 2, false, 0, false>(plan, ma, mb, mc, st);
        } else if (plan.bn == 256) s = launch<256, 1, false, 0, false>(plan, ma, mb, mc, st);
        else if (plan.bn == 192) s = launch<192, 1, false, 0, false>(plan, ma, mb, mc, st);
        else s = launch<128, 1, false, 0, false>(plan, ma, mb, mc, st);
    } else if (plan.ctas == 2) {
        if (plan.bn == 512) s = launch<512, 2>(plan, ma, mb, mc, st);
        else if (plan.bn == 384) s = launch<384, 2>(plan, ma, mb, mc, st);
        else if (plan.bn == 192) s = launch<192, 2>(plan, ma, mb, mc, st);
        else s = plan.bn == 256 ? launch<256, 2>(plan, ma, mb, mc, st) : launch<128, 2>(plan, ma, mb, mc, st);
    } else if (plan.bn == 256) s = launch<256, 1>(plan, ma, mb, mc, st);
    else if (plan.bn == 192) s = launch<192, 1>(plan, ma, mb, mc, st);
    else s = launch<128, 1>(plan, ma, mb, mc, st);
    if (s) return s;
    if (plan.p.splits > 1) {
        int64_t work = (int64_t)plan.p.batch * plan.p.M * (plan.p.N / 8);
        unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>((work + 255) / 256, (int64_t)sms * 8));
        splitk_reduce_kernel<<<grid, 256, 0, st>>>(plan.p);
        count_launch();
        CCL_CUDA_TRY(cudaGetLastError());
    }
    return CCL_OK;
}

extern "C" ccl_status ccl_gemm(const ccl_gemm_desc* d, const void* A_dev, const void* B_dev, void* C_dev, void* ws_dev,
                               size_t ws_bytes, void* cuda_stream) {
    const int64_t none[3] = {0, 0, 0};
    return gemm_impl(d, 1, false, none, A_dev, B_dev, C_dev, ws_dev, ws_bytes, cuda_stream);
}

extern "C" ccl_status ccl_gemm_batched(const ccl_gemm_desc* d, int32_t batch, const void* A_dev, int64_t a_stride_bytes, const void* B_dev,
                                       int64_t b_stride_bytes, void* C_dev, int64_t c_stride_bytes, void* ws_dev, size_t ws_bytes,
                                       void* cuda_stream) {
    if (a_stride_bytes < 0 || b_stride_bytes < 0 || c_stride_bytes < 0) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm_batched: negative stride");
    const int64_t strides[3] = {a_stride_bytes, b_stride_bytes, c_stride_bytes};
    return gemm_impl(d, batch, false, strides, A_dev, B_dev, C_dev, ws_dev, ws_bytes, cuda_stream);
}

static ccl_status grouped_impl(const ccl_gemm_desc* d, bool swiglu, int32_t groups, int64_t max_rows, const int32_t* row_offsets_dev, const void* A_dev,
                               const void* B_dev, int64_t b_stride_bytes, void* C_dev, void* cuda_stream) {
    if (!d) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm_grouped: NULL descriptor");
    if (!row_offsets_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm_grouped: NULL row offsets");
    if (reinterpret_cast<uintptr_t>(row_offsets_dev) & 3) return fail(CCL_ERR_ALIGN, "ccl_gemm_grouped: row offsets are not 4-byte aligned");
    if (max_rows < 1 || max_rows > d->M) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm_grouped: max_rows must be in [1, M]");
    if (b_stride_bytes < 0) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm_grouped: negative stride");
    if (d->a_trans) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm_grouped: A must be stored [M x K]");
    const int64_t strides[3] = {0, b_stride_bytes, 0};
    return gemm_impl(d, groups, swiglu, strides, A_dev, B_dev, C_dev, nullptr, 0, cuda_stream, 1.0f, 0.0f, row_offsets_dev, max_rows);
}

extern "C" ccl_status ccl_gemm_grouped(const ccl_gemm_desc* d, int32_t groups, int64_t max_rows, const int32_t* row_offsets_dev, const void* A_dev,
                                       const void* B_dev, int64_t b_stride_bytes, void* C_dev, void* cuda_stream) {
    return grouped_impl(d, false, groups, max_rows, row_offsets_dev, A_dev, B_dev, b_stride_bytes, C_dev, cuda_stream);
}

extern "C" ccl_status ccl_gemm_grouped_swiglu(const ccl_gemm_desc* d, int32_t groups, int64_t max_rows, const int32_t* row_offsets_dev,
                                              const void* A_dev, const void* B_dev, int64_t b_stride_bytes, void* C_dev, void* cuda_stream) {
    return grouped_impl(d, true, groups, max_rows, row_offsets_dev, A_dev, B_dev, b_stride_bytes, C_dev, cuda_stream);
}

extern "C" ccl_status ccl_gemm_grouped_k(const ccl_gemm_desc* d, int32_t groups, const int32_t* k_offsets_dev, const void* A_dev, const void* B_dev,
                                         void* C_dev, int64_t c_stride_bytes, void* cuda_stream) {
    if (!d) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm_grouped_k: NULL descriptor");
    if (!k_offsets_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm_grouped_k: NULL offsets");
    if (reinterpret_cast<uintptr_t>(k_offsets_dev) & 3) return fail(CCL_ERR_ALIGN, "ccl_gemm_grouped_k: offsets are not 4-byte aligned");
    if (c_stride_bytes < 0) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm_grouped_k: negative stride");
    const int64_t strides[3] = {0, 0, c_stride_bytes};
    return gemm_impl(d, groups, false, strides, A_dev, B_dev, C_dev, nullptr, 0, cuda_stream, 1.0f, 0.0f, nullptr, 0, k_offsets_dev);
}

extern "C" ccl_status ccl_gemm_axpby(const ccl_gemm_desc* d, float alpha, float beta, const void* A_dev, const void* B_dev, void* C_dev,
                                     void* ws_dev, size_t ws_bytes, void* cuda_stream) {
    if (!(alpha == alpha) || !(beta == beta)) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm_axpby: alpha / beta is NaN");
    const int64_t none[3] = {0, 0, 0};
    return gemm_impl(d, 1, false, none, A_dev, B_dev, C_dev, ws_dev, ws_bytes, cuda_stream, alpha, beta);
}

extern "C" ccl_status ccl_gemm_swiglu(const ccl_gemm_desc* d, const void* A_dev, const void* B_dev, void* C_dev, void* cuda_stream) {
    const int64_t none[3] = {0, 0, 0};
    return gemm_impl(d, 1, true, none, A_dev, B_dev, C_dev, nullptr, 0, cuda_stream);
}

extern "C" ccl_status ccl_gemm_status(void* cuda_stream, int32_t* detail) {
    CCL_CUDA_TRY(cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(cuda_stream)));
    int v = 0, z = 0, rv = 0;
    CCL_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_gemm_status, sizeof(int)));
    if (v) CCL_CUDA_TRY(cudaMemcpyToSymbol(g_gemm_status, &z, sizeof(int)));
    ccl_status s = repack_status_take(&rv);
    if (s) return s;
    if (detail) *detail = v ? v : (rv ? 100 + rv : 0);
    if (v == 5) return fail(CCL_ERR_SHAPE, "ccl_gemm_grouped: row offsets outside [0, M] or a problem with more rows than max_rows (such problems were not computed)");
    if (v || rv) return fail(CCL_ERR_TIMEOUT, "a bounded device-side wait expired (code %d)", v ? v : 100 + rv);
    return CCL_OK;
}

extern "C" ccl_status ccl_selftest_wait_timeout(int32_t which, uint32_t limit_us, const void* src_dev, void* cuda_stream) {
    if (which != 0 && which != 1) return fail(CCL_ERR_INVALID_ARG, "ccl_selftest_wait_timeout: which must be 0 (GEMM) or 1 (repack ring)");
    if (limit_us < 1 || limit_us > 100000) return fail(CCL_ERR_INVALID_ARG, "ccl_selftest_wait_timeout: limit_us must be in [1, 100000]");
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    const uint64_t limit_ns = (uint64_t)limit_us * 1000ull;
    if (which == 1) return repack_selftest_launch(src_dev, limit_ns, st);
    wait_selftest_kernel<<<1, 64, 0, st>>>(limit_ns);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    return CCL_OK;
}

// ------------------------------------------------------------------------------------------
// ccl_gemm_static_ws: the split-K GEMM for callers that cannot allocate
// ------------------------------------------------------------------------------------------
extern "C" ccl_status ccl_gemm_static_ws(const ccl_gemm_desc* d, const void* A_dev, const void* B_dev, void* C_dev,
                                         void* cuda_stream) {
    // (the plan -- from the prepared-call cache on every call but the first -- says how much scratch the problem needs)
    const int64_t none[3] = {0, 0, 0};
    return gemm_impl(d, 1, false, none, A_dev, B_dev, C_dev, nullptr, 0, cuda_stream, 1.0f, 0.0f, nullptr, 0, nullptr, true);
}

