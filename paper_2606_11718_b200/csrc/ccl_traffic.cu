// ccl_traffic: local / remote HBM byte counter (Sec. 4.1 metric without the L2 filter).
//
// Execution model (Sec. 2.2, Sec. 4.1): one CTA per BM x BN output tile; it reads its rows of
// A over all K, its columns of B over all K and writes its C tile.  Each operand's bytes are
// located through the operand's layout (Eq. 2 or Eq. 3), the page that holds them is mapped
// to a chiplet by the placement policy, and the bytes are local if that chiplet is the CTA's.
//
// Kernels (all integer):
//   prep      zero the outputs that are accumulated into
//   hist      per-page demand per chiplet (only when per-page output or BEST placement is asked)
//   owner     page -> chiplet for every operand whose owner table is asked for / needed
//   classify  one warp per (tile, operand): lanes walk the stored rows of the tile's rectangle,
//             cut every contiguous run at strip and page boundaries, classify, warp-reduce
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
    int64_t ntiles;
    int64_t pages[3];
    int64_t bytes_total[3];
    const int32_t* q;
    uint64_t* per_cta;
    uint64_t* per_page[3];
    uint8_t* owner[3];
    uint64_t* totals;
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
    if (p.m_strip_tiled) {
        int64_t g = tm / p.tps_m, j = tm - g * p.tps_m;
        ti.m0 = g * p.wM + j * p.BM; ti.m1 = min(ti.m0 + p.BM, (g + 1) * p.wM);
    } else { ti.m0 = tm * p.BM; ti.m1 = min(p.M, ti.m0 + p.BM); }
    if (p.n_strip_tiled) {
        int64_t g = tn / p.tps_n, j = tn - g * p.tps_n;
        ti.n0 = g * p.wN + j * p.BN; ti.n1 = min(ti.n0 + p.BN, (g + 1) * p.wN);
    } else { ti.n0 = tn * p.BN; ti.n1 = min(p.N, ti.n0 + p.BN); }
    if (p.assign == CCL_ASSIGN_N_STRIPS) ti.q = (int32_t)(ti.n0 / p.wN);
    else if (p.assign == CCL_ASSIGN_M_STRIPS) ti.q = (int32_t)(ti.m0 / p.wM);
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
            off = g * v.stride + r * v.w + (c - g * v.w);
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

constexpr int kWarpsPerBlock = 8;

__global__ void __launch_bounds__(kWarpsPerBlock * 32) traffic_hist_kernel(TrafficParams p) {
    const int lane = threadIdx.x & 31;
    const int64_t nwork = p.ntiles * 3;
    for (int64_t wk = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5); wk < nwork; wk += (int64_t)gridDim.x * kWarpsPerBlock) {
        int64_t t = wk / 3;
        int X = (int)(wk - t * 3);
        if (!p.per_page[X]) continue;
        TileInfo ti = decode_tile(p, t);
        int64_t r0, r1, c0, c1;
        tile_rect(p, ti, X, r0, r1, c0, c1);
        unsigned long long* hist = reinterpret_cast<unsigned long long*>(p.per_page[X]);
        for (int64_t r = r0 + lane; r < r1; r += 32)
            walk_row(p, p.v[X], r, c0, c1, [&](int64_t page, int64_t len) { atomicAdd(&hist[page * p.P + ti.q], (unsigned long long)len); });
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

__global__ void __launch_bounds__(kWarpsPerBlock * 32) traffic_classify_kernel(TrafficParams p) {
    __shared__ unsigned long long blk[6];
    if (threadIdx.x < 6) blk[threadIdx.x] = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int64_t nwork = p.ntiles * 3;
    for (int64_t wk = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5); wk < nwork; wk += (int64_t)gridDim.x * kWarpsPerBlock) {
        int64_t t = wk / 3;
        int X = (int)(wk - t * 3);
        TileInfo ti = decode_tile(p, t);
        int64_t r0, r1, c0, c1;
        tile_rect(p, ti, X, r0, r1, c0, c1);
        unsigned long long loc = 0, rem = 0;
        const bool table = p.place[X] == CCL_PLACE_BEST;
        const uint8_t* own = p.owner[X];
        for (int64_t r = r0 + lane; r < r1; r += 32)
            walk_row(p, p.v[X], r, c0, c1, [&](int64_t page, int64_t len) {
                int32_t o = table ? (int32_t)own[page] : fixed_owner(p, X, page);
                if (o == ti.q) loc += (unsigned long long)len; else rem += (unsigned long long)len;
            });
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) {
            loc += __shfl_xor_sync(0xffffffffu, loc, s);
            rem += __shfl_xor_sync(0xffffffffu, rem, s);
        }
        if (lane == 0) {
            p.per_cta[t * 6 + X * 2 + 0] = loc;
            p.per_cta[t * 6 + X * 2 + 1] = rem;
            atomicAdd(&blk[X * 2 + 0], loc);
            atomicAdd(&blk[X * 2 + 1], rem);
        }
    }
    __syncthreads();
    if (threadIdx.x < 6 && blk[threadIdx.x]) atomicAdd(reinterpret_cast<unsigned long long*>(p.totals) + threadIdx.x, blk[threadIdx.x]);
}

static ccl_status fill_params(const ccl_traffic_desc* d, TrafficParams* p) {
    if (!d) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic: NULL descriptor");
    std::memset(p, 0, sizeof(*p));
    if (d->M <= 0 || d->N <= 0 || d->K <= 0 || d->BM <= 0 || d->BN <= 0) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic: sizes must be positive");
    if (d->P < 1 || d->P > 255) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic: P must be in [1,255]");
    if (d->page_bytes <= 0) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic: page_bytes must be positive");
    if (d->assign < 0 || d->assign > 2) return fail(CCL_ERR_INVALID_ARG, "ccl_traffic: unknown assign");
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
    if (d->assign == CCL_ASSIGN_N_STRIPS && d->N % d->P) return fail(CCL_ERR_SHAPE, "ccl_traffic: N not divisible by P");
    if (d->assign == CCL_ASSIGN_M_STRIPS && d->M % d->P) return fail(CCL_ERR_SHAPE, "ccl_traffic: M not divisible by P");
    p->M = d->M; p->N = d->N; p->K = d->K; p->BM = d->BM; p->BN = d->BN;
    p->a_trans = d->a_trans != 0; p->b_trans = d->b_trans != 0; p->P = d->P; p->S = d->page_bytes;
    p->s_shift = -1;
    if ((d->page_bytes & (d->page_bytes - 1)) == 0) { int sh = 0; while ((INT64_C(1) << sh) < d->page_bytes) ++sh; p->s_shift = sh; }
    p->assign = d->assign;
    p->m_strip_tiled = d->assign == CCL_ASSIGN_M_STRIPS && d->strip_tiling;
    p->n_strip_tiled = d->assign == CCL_ASSIGN_N_STRIPS && d->strip_tiling;
    p->wM = d->assign == CCL_ASSIGN_M_STRIPS ? d->M / d->P : d->M;
    p->wN = d->assign == CCL_ASSIGN_N_STRIPS ? d->N / d->P : d->N;
    p->tps_m = p->m_strip_tiled ? (p->wM + d->BM - 1) / d->BM : 0;
    p->tps_n = p->n_strip_tiled ? (p->wN + d->BN - 1) / d->BN : 0;
    p->tiles_m = p->m_strip_tiled ? p->tps_m * d->P : (d->M + d->BM - 1) / d->BM;
    p->tiles_n = p->n_strip_tiled ? p->tps_n * d->P : (d->N + d->BN - 1) / d->BN;
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

    int64_t nwork = p.ntiles * 3;
    unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>((nwork + kWarpsPerBlock - 1) / kWarpsPerBlock, (int64_t)sms * 8));
    if (need_hist) {
        traffic_hist_kernel<<<grid, kWarpsPerBlock * 32, 0, st>>>(p);
        count_launch();
        CCL_CUDA_TRY(cudaGetLastError());
    }
    if (need_owner) {
        traffic_owner_kernel<<<sms * 2, 256, 0, st>>>(p);
        count_launch();
        CCL_CUDA_TRY(cudaGetLastError());
    }
    traffic_classify_kernel<<<grid, kWarpsPerBlock * 32, 0, st>>>(p);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    return CCL_OK;
}
