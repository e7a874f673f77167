// Host-side planning of a GEMM call: operand checks, the choice of kernel variant (tile shape, CTA pairing, K splits, cluster
// split, balanced split) from a cost model built on measured per-block figures, the parameter block and the tensor maps.
// Included by ccl_gemm.cu only, after ccl_gemm_kernel.cuh.
#ifndef CCL_GEMM_PLAN_CUH_
#define CCL_GEMM_PLAN_CUH_

#include "ccl_gemm_kernel.cuh"

namespace ccl {

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
struct GemmPlan {
    GemmParams p;
    int bn, ctas, subn;
    int a_box_rows;            // rows of A's TMA box (BM unless A has fewer than 8 rows)
    CUtensorMap ma2, mb2, mc2; // the last strips of operands whose strips are not all alike (else copies of the operands' maps)
    size_t ws_bytes;
    MatView va, vb, vc;
    uint32_t smem_bytes;
    bool lean;                 // no optional feature in use (see FULL)
    unsigned grid;
    int ks;                    // cluster split along K: CTAs per cluster (0: none)
};

// How a page-interleaved operand is expressed as a rank-4 tensor map (OpMap::il_mode): 0 = not interleaved,
// 1 = a chunk holds *kr whole strip rows, 2 = a strip row spans whole chunks, -1 = neither (no affine map exists).
static int interleave_mode(const MatView& v, int64_t* kr) {
    *kr = 0;
    if (!v.ichunk) return 0;
    const int64_t row = v.split == 2 ? v.w : v.cols;
    if (v.ichunk % row == 0) { *kr = v.ichunk / row; return 1; }
    if (row % v.ichunk == 0 && v.ichunk % 64 == 0) return 2;
    if (row % 64 == 0 && v.ichunk % 64 == 0) return 3;      // no affine box, but every 128-byte piece of a row lies inside one chunk
    return -1;
}

// k_along_rows: the GEMM's K dimension runs along the stored rows of this operand (never for C)
static ccl_status check_operand(const MatView& v, const void* ptr, const char* name, bool k_along_rows, int64_t K, bool is_c = false) {
    if (v.e != 2) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: only 2-byte (bf16) elements are supported", name);
    if (ragged(v)) {                     // a last strip narrower / lower than the others: it gets a tensor map of its own
        if (v.ichunk) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: a page-interleaved operand with strips of unequal size is not supported", name);
        if (!is_c && (k_along_rows ? v.split == 1 : v.split == 2))
            return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: strips of unequal size along K are not supported", name);
        if (v.split == 2 && v.wlast % 8) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: the last strip's %lld columns are not a multiple of 8", name, (long long)v.wlast);
    }
    int64_t inner = v.split == 2 ? v.w : v.cols;
    if (inner % 8) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: contiguous extent %lld is not a multiple of 8 elements", name, (long long)inner);
    if (v.ichunk) {
        int64_t kr;
        const int mode = interleave_mode(v, &kr);
        if (mode < 0)
            return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: page-interleaved layout: a chunk (%lld elements) must hold whole strip rows (%lld elements), "
                        "or a strip row whole chunks of a multiple of 64 elements, or both must be multiples of 64 elements", name, (long long)v.ichunk, (long long)inner);
        if (mode == 3) {                     // fetched row by row (see line_of): what that path assumes
            if (k_along_rows ? v.split == 1 : (v.split == 2 && !is_c))
                return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: a page-interleaved operand whose chunks and strip rows do not line up must not be split along K", name);
            if (!k_along_rows && !is_c && K % BK)
                return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: page-interleaved layout: K (%lld) must be a multiple of %d when chunks and strip rows do not line up", name, (long long)K, BK);
            if ((double)(v.split == 1 ? v.h : v.rows) * (double)inner >= 2147483648.0 || buffer_elems(v) / 64 >= (INT64_C(1) << 31))
                return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: strip too large for the row-by-row path", name);
        }
        if (mode == 1 && (kr & (kr - 1)))
            return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: page-interleaved layout: %lld strip rows per chunk is not a power of two", name, (long long)kr);
        const int64_t R = v.split == 1 ? v.h : v.rows;
        // rows past the strip's end inside its last chunk are padding, not zeros: a ragged K tail must not read them
        if (mode == 1 && k_along_rows && K % BK && R % kr)
            return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: page-interleaved layout: K (%lld) is not a multiple of %d and ends inside a chunk", name, (long long)K, BK);
        if ((v.ichunk * v.e) % 16) return fail(CCL_ERR_ALIGN, "ccl_gemm: %s: chunk size is not a multiple of 16 bytes", name);
        if ((double)v.nstrips * (double)std::max(v.ichunk, inner) * v.e >= (double)(INT64_C(1) << 40))
            return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: extent too large for a tensor map", name);
    } else if (v.split && (v.stride * v.e) % 16) return fail(CCL_ERR_ALIGN, "ccl_gemm: %s: strip stride is not a multiple of 16 bytes", name);
    if (ptr && (reinterpret_cast<uintptr_t>(ptr) & 15)) return fail(CCL_ERR_ALIGN, "ccl_gemm: %s: base pointer is not 16-byte aligned", name);
    if (v.rows >= (INT64_C(1) << 31) || v.cols >= (INT64_C(1) << 31) || v.stride * v.e >= (INT64_C(1) << 40))
        return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: %s: extent too large for a tensor map", name);
    return CCL_OK;
}

// strip width an operand imposes on the GEMM dimension that runs along its stored rows / cols
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

// units = schedulable CTAs (1-CTA kernel) or CTA pairs (2-CTA kernel) the device can hold at once
// cap > 0: a ragged batch -- the tile grid of one problem covers `cap` rows, d->M is the total row count of A and C
// ragk: a batch with ragged K -- d->K is the total row count of the concatenated A [K x M] and B [K x N]
static int resident_clusters(int ks, bool have_device);

// Modelled cycles of one k block (64 of K) of a tile `b` columns wide on `c` CTAs: the tensor pipe needs 2 cycles per tile
// column (128 rows per SM, UMMA_K = 16, four steps); the SM pulls its share of the operands (its 128 rows of A and its
// columns of B, whole 64-column boxes of an N-contiguous B) from the L2 at ~70 B/clk on its own and at its share of
// ~9 KB/clk when `active` CTAs pull at once (61 B/clk with all 148: 128 x 192 tiles measured 670 cycles per block in a
// batch that fills the machine, 585 alone); the producer and MMA-issue loops need ~450 cycles per block whatever the
// tile (all measured with per-role timestamps); the longest of the three, plus the hand-over.
static double kblock_cycles(int b, int c, bool b_kmajor, int64_t active) {
    const double b_cols = (double)(b_kmajor ? b / c : (b / c + 63) / 64 * 64);
    const double rate = std::min(70.0, 9000.0 / (double)std::max<int64_t>(1, active));
    return std::max(std::max(2.0 * b, (BM + b_cols) * (BK * 2) / rate), 450.0) + 15.0;
}

// have_device: the unit counts come from the current device (else the figures of a B200)
static ccl_status make_plan(const ccl_gemm_desc* d, int64_t batch, bool swiglu, const void* A, const void* B, const void* C, int sms, int pairs, GemmPlan* plan,
                            int64_t cap = 0, bool ragk = false, size_t max_ws = ~(size_t)0, bool have_device = false) {
    if (!d) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm: NULL descriptor");
    if (d->M <= 0 || d->N <= 0 || d->K <= 0) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm: M, N, K must be positive");
    if (d->M >= (INT64_C(1) << 31) || d->N >= (INT64_C(1) << 31) || d->K >= (INT64_C(1) << 31)) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: dimension too large");
    if (d->out_part < 0 || d->out_part > 3) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm: unknown out_part");
    if (d->out_part == CCL_PART_2D && (d->part_m < 1 || d->P % d->part_m)) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm: part_m (%d) must divide P (%d)", d->part_m, d->P);
    if (d->out_part == CCL_PART_2D && swiglu) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm_swiglu: a 2-D output partition is not supported");
    if (d->P < 1 || d->P > 255) return fail(CCL_ERR_INVALID_ARG, "ccl_gemm: P must be in [1,255]");
    ccl_status s;
    if ((s = make_view(&d->A, "ccl_gemm: A", &plan->va))) return s;
    if ((s = make_view(&d->B, "ccl_gemm: B", &plan->vb))) return s;
    if ((s = make_view(&d->C, "ccl_gemm: C", &plan->vc))) return s;
    const MatView &va = plan->va, &vb = plan->vb, &vc = plan->vc;
    const bool at = d->a_trans != 0, bt = d->b_trans != 0;
    int64_t ar = at ? d->K : d->M, ac = at ? d->M : d->K, br = bt ? d->N : d->K, bc = bt ? d->K : d->N;
    if (swiglu && d->N % 2) return fail(CCL_ERR_SHAPE, "ccl_gemm_swiglu: N (gate + up columns) must be even");
    const int64_t Nc = swiglu ? d->N / 2 : d->N;        // columns of C, which the tile walk counts
    if (va.rows != ar || va.cols != ac || vb.rows != br || vb.cols != bc || vc.rows != d->M || vc.cols != Nc)
        return fail(CCL_ERR_SHAPE, "ccl_gemm: operand shapes do not match M, N, K and the transpose flags");
    if (swiglu && (va.ichunk || vb.ichunk || vc.ichunk))
        return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm_swiglu: page-interleaved operands are not supported");
    if ((s = check_operand(va, A, "A", at, d->K))) return s;
    if ((s = check_operand(vb, B, "B", !bt, d->K))) return s;
    if ((s = check_operand(vc, C, "C", false, d->K, true))) return s;
    int64_t kr_a, kr_b, kr_c;
    const int il_a = interleave_mode(va, &kr_a), il_b = interleave_mode(vb, &kr_b), il_c = interleave_mode(vc, &kr_c);
    if ((il_a == 3 || il_b == 3 || il_c == 3) && (batch > 1 || cap > 0 || ragk))
        return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: a batch with a page-interleaved operand whose chunks and strip rows do not line up is not supported");
    // a 192-row (96-row for a CTA pair) box of a K-contiguous B cannot be cut into chunks of more than 64 (32) rows
    const bool no_192 = il_b == 1 && bt && kr_b > 64, no_192_pair = il_b == 1 && bt && kr_b > 32;

    // strips along M, N (tiles must not straddle them) and along K (a 64-wide k block must not)
    int64_t Wm = 0, Wn = 0;
    if ((s = merge_width(&Wm, split_width(va, !at), "M"))) return s;
    if ((s = merge_width(&Wm, split_width(vc, true), "M"))) return s;
    if (swiglu) {
        // a strip of B holds the gate and the up columns of one strip of C: twice as wide
        const int64_t wb = split_width(vb, bt);
        if (wb % 2) return fail(CCL_ERR_SHAPE, "ccl_gemm_swiglu: strips of B have an odd width");
        if ((s = merge_width(&Wn, wb / 2, "N"))) return s;
        // the gate | up halves follow the output partition whether or not the raster is grouped
        if (d->out_part == CCL_PART_COLS && d->P > 1) {
            if (Nc % d->P) return fail(CCL_ERR_SHAPE, "ccl_gemm_swiglu: N/2 not divisible by P");
            if ((s = merge_width(&Wn, Nc / d->P, "N"))) return s;
        }
    } else if ((s = merge_width(&Wn, split_width(vb, bt), "N"))) return s;
    if ((s = merge_width(&Wn, split_width(vc, false), "N"))) return s;
    int groups = 1, group_dim = 0, groups_n = 1;
    if (d->grouped_raster && d->P > 1 && d->out_part != CCL_PART_NONE) {
        if (d->out_part == CCL_PART_2D) {                 // part_m x (P / part_m) blocks of the output, one CTA group each
            const int pm = d->part_m, pn = d->P / d->part_m;
            if (d->M % pm || Nc % pn) return fail(CCL_ERR_SHAPE, "ccl_gemm: M / N not divisible by the %d x %d output partition", pm, pn);
            if (pm > 1 && (s = merge_width(&Wm, d->M / pm, "M"))) return s;
            if (pn > 1 && (s = merge_width(&Wn, Nc / pn, "N"))) return s;
            groups = d->P; group_dim = 2; groups_n = pn;
        } else if (d->out_part == CCL_PART_COLS) {
            // (N not a multiple of P: the strips are those of the operands -- ceil(N / P) wide, the last one narrower)
            if (Nc % d->P) { if (!(Wn > 0 && (Nc + Wn - 1) / Wn == d->P)) return fail(CCL_ERR_SHAPE, "ccl_gemm: N not divisible by P"); }
            else if ((s = merge_width(&Wn, Nc / d->P, "N"))) return s;
            groups = d->P; group_dim = 0;
        } else {
            if (d->M % d->P) { if (!(Wm > 0 && (d->M + Wm - 1) / Wm == d->P)) return fail(CCL_ERR_SHAPE, "ccl_gemm: M not divisible by P"); }
            else if ((s = merge_width(&Wm, d->M / d->P, "M"))) return s;
            groups = d->P; group_dim = 1;
        }
    }
    int64_t ka = split_width(va, at), kb = split_width(vb, !bt);
    if ((ka && ka % BK) || (kb && kb % BK)) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: an operand split along K needs strips that are multiples of %d", BK);
    if (ragk && (!at || bt || ka || kb || il_a || il_b))
        return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm_grouped_k: A must be stored [K x M] and B [K x N], neither split along K nor page-interleaved");
    const bool any_rag = ragged(va) || ragged(vb) || ragged(vc);
    if (any_rag && (batch > 1 || cap > 0 || ragk || swiglu || d->out_part == CCL_PART_2D))
        return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: strips of unequal size are taken by the plain call only (no batch, fused activation or 2-D partition)");
    const int64_t Mt = cap > 0 ? cap : d->M;            // rows the tile grid of one problem covers
    if (cap > 0 && Wm) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm_grouped: A and C must not be split along M");
    if (!Wm) Wm = Mt;
    if (!Wn) Wn = Nc;
    if (swiglu) {
        const int64_t pd = d->out_part == CCL_PART_COLS && d->P > 1 ? Nc / d->P : Nc;      // gate -> up distance in B
        if (Wn != pd) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm_swiglu: strips of B / C (%lld output columns) differ from the gate | up halves (%lld)", (long long)Wn, (long long)pd);
        if (pd % 8) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm_swiglu: gate | up halves of %lld columns are not a multiple of 8", (long long)pd);
        if (pairs <= 0) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm_swiglu: needs 2-CTA clusters");
    }

    // Tile shape, CTA pairing and split-K from a small cost model (cycles per unit):
    //   a k block of a one-accumulator tile takes ~600 cycles whatever its width (four MMAs are issued in ~350
    //   cycles and the barrier round trip adds ~250), a 256 x 512 pair tile ~1050 (its eight MMAs keep the
    //   tensor pipe busy for 1024); a tile that nobody shares its B columns with (one row of tiles) streams
    //   them from HBM at this SM's share of the bandwidth, ~27 B/clk;
    //   a one-accumulator tile hides its drain behind the next tile's main loop (TMEM double buffer), the wide
    //   tile exposes it (~7000 cycles); split-K adds the partial-sum traffic and a second launch.
    // 256 x 512 pair tiles move the fewest bytes per flop and win once K is long; short problems prefer the
    // variant whose tile count fills the machine.
    const int64_t num_kb = ((ragk ? std::max<int64_t>(1, d->K / batch) : d->K) + BK - 1) / BK;   // (ragged K: the mean, for the cost model only)
    const int64_t strips_m = (Mt + Wm - 1) / Wm, strips_n = (Nc + Wn - 1) / Wn;
    // a tile starts at a multiple of the strip width: where that is the contiguous coordinate of a tensor map -- the columns of
    // C (and of an N-contiguous B), the columns of an A stored [K x M] -- it must be a multiple of 8 elements (16 bytes)
    if (strips_n > 1 && Wn % 8) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: strips of %lld columns of N are not a multiple of 8", (long long)Wn);
    if (strips_m > 1 && at && Wm % 8) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: strips of %lld columns of an A stored [K x M] are not a multiple of 8", (long long)Wm);
    int ctas = 1, bn = 256, splits = 1;
    double best = -1.0;
    // Test overrides (environment): CCL_GEMM_CTAS = 1|2, CCL_GEMM_BN = 128|192|256|384|512, CCL_GEMM_SPLITK = number of K splits.
    const char* force_ctas = std::getenv("CCL_GEMM_CTAS");
    const char* force_bn = std::getenv("CCL_GEMM_BN");
    const char* force_split = std::getenv("CCL_GEMM_SPLITK");
    for (int c = 1; c <= 2; ++c) {
        if (c == 2 && (pairs <= 0 || ragk)) continue;          // (a ragged-K tail is zeroed by the CTA that issues the MMAs)
        if (force_ctas && atoi(force_ctas) != c) continue;
        const int units = c == 2 ? pairs : sms;
        for (int b : {512, 384, 256, 192, 128}) {
            if (c == 1 && b > 256) continue;
            if (c == 2 && b == 192 && !bt && il_b) continue;    // 96 columns per CTA of an N-contiguous B: a box and a half (see the kernel), not across chunks
            if (b == 192 && (c == 2 ? no_192_pair : no_192)) continue;
            if (b == 384 && (cap > 0 || ragk)) continue;            // (no ragged-batch instantiation of the 256 + 128 tile)
            if (force_bn && atoi(force_bn) != b) continue;
            if (swiglu && !(c == 2 && b == 512)) continue;          // the gated activation pairs the two accumulators of the wide tile
            const int64_t tiles_m_all = strips_m * ((Wm + BM * c - 1) / (BM * c));
            const int bs = swiglu ? 256 : b;                        // tile width in C columns
            const int64_t tiles = tiles_m_all * strips_n * ((Wn + bs - 1) / bs) * batch;
            // a k block: the tensor pipe needs 2 cycles per tile column (128 rows per SM, UMMA_K = 16, four steps), the
            // SM pulls its share of the operands (its 128 rows of A and its columns of B, whole 64-column boxes of an
            // N-contiguous B) from the L2 at ~70 B/clk; whichever is longer, plus the hand-over
            const double t_kb = kblock_cycles(b, c, bt, std::min<int64_t>(tiles, units) * c);
            const double t_drain = b == 512 ? 7000.0 : (b == 384 ? 5500.0 : 1500.0);
            // one row of tiles: nobody shares the B columns, the problem streams B from HBM at ~29 B/clk per SM in
            // aggregate however the units are cut (a ragged last wave still saturates the memory); wider boxes are
            // fetched a little more efficiently (measured: 128 / 192 columns cost ~10 % / ~4 % more time per byte)
            const double stream_clk = tiles_m_all == 1 ? (double)tiles * (double)num_kb * (double)b * (BK * 2) / (sms * 29.0) *
                                                             (b <= 128 ? 1.10 : (b <= 192 ? 1.04 : 1.0)) : 0.0;
            for (int sp : {1, 2, 3, 4, 6, 8, 12, 16}) {
                if (sp > 1 && (swiglu || cap > 0 || ragk || any_rag || num_kb / sp < 2)) continue;
                if (force_split && atoi(force_split) != sp) continue;
                const int64_t kbps = (num_kb + sp - 1) / sp;
                const int64_t sp_eff = (num_kb + kbps - 1) / kbps;          // every split owns at least one k block
                if (sp_eff != sp) continue;
                const int64_t waves = (tiles * sp + units - 1) / units;
                // (a last wave that leaves SMs idle streams a little slower: measured ~5 % between 96 and 128 busy SMs)
                const double last = (double)(tiles * sp - (waves - 1) * units) / (double)units;
                double cost = std::max((double)waves * ((double)kbps * t_kb + (sp > 1 ? 2.0 * t_drain : t_drain)),
                                       stream_clk * (1.0 + 0.1 * (1.0 - last))) + 3000.0;
                // a problem that runs for long runs at the power cap, where the clock follows the energy a k block costs:
                // measured, 256 x 256 pair tiles (a third more operand bytes per flop than 256 x 512) take 3-6 % longer on
                // the Llama-size GEMMs although they need fewer cycles
                if (cost > 3.0e5) cost *= 1.0 + 0.25 * ((BM + (double)b / c) / ((double)b / c) / 1.5 - 1.0);
                if (sp > 1) cost += ((double)sp + 0.5) * (double)batch * (double)Mt * (double)d->N * 4.0 / 3400.0 + 14000.0;
                if (best < 0 || cost < best) { best = cost; ctas = c; bn = b; splits = sp; }
            }
        }
    }
    if (best < 0) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: no kernel variant matches the forced CCL_GEMM_* settings");
    // Balanced split: instead of whole tiles, every unit of a group gets the same number of k blocks of the group's tiles
    // laid end to end (at most `share`), so nothing is lost to a last round that fills a fraction of the machine or to a
    // tile count below the unit count.  A tile cut between units costs one unit its partial sums (written to the
    // workspace while its next tile computes) and the finishing unit a read of them; with shares shorter than a tile the
    // shares of a tile run side by side and the finishing one reads several.  Modelled in the same cycles as above.
    bool balanced = false;
    {
        const char* force_bal = std::getenv("CCL_GEMM_BALANCED");   // 0: never, 1: whenever the call qualifies
        const int want = force_bal ? atoi(force_bal) : -1;
        const bool can = want != 0 && batch == 1 && !swiglu && cap == 0 && !ragk && !any_rag && num_kb >= 2 && !(force_split && atoi(force_split) > 1);
        double best_bal = -1.0;
        int bc = 0, bb = 0;
        int64_t bal_rounds = 0;
        for (int c = 1; can && c <= 2; ++c) {
            if (c == 2 && pairs <= 0) continue;
            if (force_ctas && atoi(force_ctas) != c) continue;
            const int units = c == 2 ? pairs : sms;
            for (int b : {512, 256, 192, 128}) {
                if (c == 1 && b > 256) continue;
                if (c == 2 && b == 192 && !bt) continue;
                if (b == 192 && (c == 2 ? no_192_pair : no_192)) continue;
                if (force_bn && atoi(force_bn) != b) continue;
                const int64_t tm = strips_m * ((Wm + BM * c - 1) / (BM * c)), tn = strips_n * ((Wn + b - 1) / b);
                if (tm == 1 && want != 1) continue;              // one row of tiles streams B from HBM: the split-K plans above are tuned for it
                int G = 1;
                if (groups > 1 && units >= groups && (group_dim == 0 ? tn % groups == 0 : group_dim == 1 ? tm % groups == 0
                                                                    : (tn % groups_n == 0 && tm % (groups / groups_n) == 0))) G = groups;
                const int64_t tiles_g = tm * tn / G;
                const int upg = units / G;
                const int64_t rounds = tiles_g / upg, rest = tiles_g - rounds * upg;     // whole rounds, tiles of the shared part
                if (rest == 0 || rest * num_kb >= (INT64_C(1) << 30)) continue;
                const int64_t sharers = std::max<int64_t>(1, std::min<int64_t>(upg, rest * num_kb / 4));   // a share is at least four k blocks
                const int64_t share = (rest * num_kb + sharers - 1) / sharers;
                const size_t ws = (size_t)G * upg * c * 2 * ((size_t)BM * b * 4 + 32);
                if (ws > max_ws) continue;
                const double t_kb = b == 512 ? 1050.0 : (c == 1 && b == 256 ? 680.0 : (c == 1 ? 570.0 : 620.0));
                const double t_drain = b == 512 ? 7000.0 : 1500.0;
                // every sharer writes its partial sums and reads as much back (its part of the columns from every
                // sharer), all of them at the same time: measured ~17 B/clk per SM then (the L2's write side saturates);
                // this runs behind the unit's next tile if it has one (costing that tile a little of its operand
                // bandwidth), and is the tail of the kernel if the shares are all there is
                const double fix = 2.0 * (double)BM * b * 4 / 17.0;
                const double cost = ((double)share + (double)rounds * num_kb) * t_kb + t_drain + (rounds == 0 ? fix : 0.15 * fix) + 3000.0 + 2500.0;
                if (best_bal < 0 || cost < best_bal) { best_bal = cost; bc = c; bb = b; bal_rounds = rounds; }
            }
        }
        // Measured (B200): on its own the planner never takes it.  Short GEMMs lose more to the partial-sum traffic (fp32
        // through the L2, whose write side all sharers hit at once: ~17 B/clk per SM) and to the extra node in front of the
        // launch than they gain (Qwen-size shapes: 1.2-2x slower), and a long GEMM runs at the power cap, where fewer idle
        // cycles come back as lower clocks, not less time (4096 x 8192 x 8192: 9 % fewer cycles, 1 % less time; the two
        // benchmark GEMMs: 2-3 % more time, for the two CTA pairs the equal groups leave out).  CCL_GEMM_BALANCED=1 turns it
        // on wherever it is legal.
        if (best_bal > 0 && want == 1) { ctas = bc; bn = bb; splits = 1; balanced = true; best = best_bal; }
        (void)bal_rounds;                                   // (kept in the model for the record)
    }
    // Cluster split: a problem of few tiles and a long K -- fewer tiles than a fraction of the SMs -- is split along K
    // inside a cluster of 2, 4 or 8 CTAs per 128 x BN tile, the partial sums meeting in distributed shared memory: no
    // workspace, no second launch.  No batch, fused activation, page-interleaved or K-split operand; CCL_GEMM_CLUSTERK = 0 turns it off, = 2|4|8 forces the cluster size.
    int ks = 0;
    {
        const char* force_ks = std::getenv("CCL_GEMM_CLUSTERK");
        const int want_ks = force_ks ? atoi(force_ks) : -1;
        const bool can = want_ks != 0 && batch == 1 && !swiglu && cap == 0 && !ragk && !any_rag && !il_a && !il_b && !il_c && !ka && !kb &&
                         !(force_split && atoi(force_split) > 1) && !balanced && !(force_ctas && atoi(force_ctas) != 1) && d->out_part != CCL_PART_2D;
        double best_ks = -1.0;
        int kb_ = 0, kk = 0;
        for (int b : {256, 192, 128}) {
            if (!can) break;
            if (b == 192 && no_192) continue;
            if (force_bn && atoi(force_bn) != b) continue;
            const int64_t tiles = strips_m * ((Wm + BM - 1) / BM) * strips_n * ((Wn + b - 1) / b);
            for (int k : {2, 4, 8}) {
                if (want_ks > 0 && want_ks != k) continue;
                if (tiles > resident_clusters(k, have_device) || tiles * k > sms) continue;
                const int64_t kbps = (num_kb + k - 1) / k;
                if ((num_kb + kbps - 1) / kbps != k || kbps < 2) continue;           // every CTA of the cluster owns k blocks
                // drain, the exchange (every CTA sends (k - 1) / k of its sums and adds up k sources: ~1000 cycles per CTA of
                // the cluster, measured on 256 x 768 x 2048: 7.0 / 7.4 / 7.9 / 8.5 us with clusters of 4 / 3 / 6 / 8), launch
                const double cost = (double)kbps * kblock_cycles(b, 1, bt, tiles * k) + 1500.0 + (1000.0 + 1000.0 * k) + 3000.0;
                if (best_ks < 0 || cost < best_ks) { best_ks = cost; kb_ = b; kk = k; }
            }
        }
        if (best_ks > 0 && (want_ks > 0 || best_ks < 0.95 * best)) { ctas = 1; bn = kb_; splits = 1; ks = kk; best = best_ks; }
    }
    if (std::getenv("CCL_GEMM_VERBOSE"))
        std::fprintf(stderr, "ccl_gemm plan: %lld x %lld x %lld batch %lld -> %d CTA(s) per tile, tile width %d, %d K split(s)%s, modelled %.0f cycles\n",
                     (long long)d->M, (long long)d->N, (long long)d->K, (long long)batch, ctas, bn, splits, balanced ? ", balanced split" : (ks ? ", cluster split along K" : ""), best);
    const int subn = bn > 256 ? 256 : bn;                // columns of one MMA / one TMEM accumulator
    plan->subn = subn;
    const int bm = BM * ctas;
    plan->bn = bn; plan->ctas = ctas;
    plan->ws_bytes = splits > 1 ? (size_t)batch * (size_t)splits * (size_t)d->M * (size_t)d->N * 4 : 0;

    GemmParams& p = plan->p;
    std::memset(&p, 0, sizeof(p));
    p.M = (int32_t)d->M; p.N = (int32_t)Nc; p.K = (int32_t)d->K;
    const int bn_walk = swiglu ? 256 : bn;              // tile width in C columns
    p.pair_dist = swiglu ? (int32_t)Wn : 0; p.fd_wn = make_fastdiv(Wn);
    p.Wm = (int32_t)Wm; p.Wn = (int32_t)Wn;
    p.tps_m = (int32_t)((Wm + bm - 1) / bm); p.tps_n = (int32_t)((Wn + bn_walk - 1) / bn_walk);
    p.tiles_m = (int32_t)((Mt + Wm - 1) / Wm) * p.tps_m; p.tiles_n = (int32_t)((Nc + Wn - 1) / Wn) * p.tps_n;
    p.num_kb = (int32_t)num_kb;
    p.splits = splits; p.kb_per_split = (int32_t)((num_kb + splits - 1) / splits);
    p.a.split = va.split; p.a.w = make_fastdiv(va.w); p.a.h = make_fastdiv(va.h);
    p.b.split = vb.split; p.b.w = make_fastdiv(vb.w); p.b.h = make_fastdiv(vb.h);
    p.a_mn = at ? 1 : 0; p.b_mn = bt ? 0 : 1;
    p.a.il_mode = il_a; p.a.il_kr = make_fastdiv(kr_a); p.a.il_sc = make_fastdiv(va.ichunk);
    p.b.il_mode = il_b; p.b.il_kr = make_fastdiv(kr_b); p.b.il_sc = make_fastdiv(vb.ichunk);
    p.c.split = vc.split; p.c.w = make_fastdiv(vc.w); p.c.h = make_fastdiv(vc.h);
    p.c.il_mode = il_c; p.c.il_kr = make_fastdiv(kr_c); p.c.il_sc = make_fastdiv(vc.ichunk);
    {
        const MatView* vs[3] = {&va, &vb, &vc};
        OpMap* os[3] = {&p.a, &p.b, &p.c};
        for (int X = 0; X < 3; ++X) {
            os[X]->rows = (int32_t)vs[X]->rows; os[X]->cols = (int32_t)vs[X]->cols;
            os[X]->roww = (int32_t)(vs[X]->split == 2 ? vs[X]->w : vs[X]->cols); os[X]->nstrips = (int32_t)vs[X]->nstrips;
            os[X]->lines = os[X]->il_mode == 3 ? (int32_t)(buffer_elems(*vs[X]) / 64) : 0;
            os[X]->rag = ragged(*vs[X]) ? 1 : 0;
        }
    }
    p.c_row = vc.split == 2 ? vc.w : vc.cols; p.c_stride = vc.stride;
    p.c_wlast = ragged(vc) && vc.split == 2 ? (int32_t)vc.wlast : 0;
    p.c_ichunk = vc.ichunk; p.c_nstrips = vc.nstrips;
    p.c_cpr = il_c == 2 ? (int32_t)(p.c_row / vc.ichunk) : 0;
    // instruction descriptor: D = f32, A = B = bf16, operand majors, N >> 3, M >> 4 (M spans the CTA pair)
    p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.a_mn << 15) | ((uint32_t)p.b_mn << 16) |
              ((uint32_t)(subn >> 3) << 17) | ((uint32_t)(bm >> 4) << 24);
    // Fewer than 8 rows of a K-contiguous A (a decode step): the box holds just those rows.  Measured, a 128-row box of
    // which fewer than one 8-row swizzle group exists makes the weight-streaming GEMM 57344 x 8192 take 170 us at
    // M = 1 ... 7 against 147 us at M = 8 ... 33.  The rows of the stage the box no longer writes keep what was there:
    // they only feed accumulator rows past M, which no epilogue stores.
    plan->a_box_rows = (!at && cap == 0 && !ragk && !il_a && d->M < 8) ? (int)d->M : BM;
    p.a_bytes = BM * BK * 2; p.stage_bytes = p.a_bytes + (uint32_t)(p.b_mn ? (bn / ctas + 63) / 64 * 64 : bn / ctas) * BK * 2;   // (an N-contiguous B comes in whole 64-column boxes)
    // a ragged batch of up to kRaggedDense problems walks only real tiles: the prefix of their tile counts sits behind
    // the barriers in shared memory, and the operand ring gives up that room
    // (CCL_GEMM_RAGGED_DENSE=0: the fixed grid of max_rows per problem with empty tiles skipped, as for larger batches)
    p.tx_bytes = p.stage_bytes - (uint32_t)(BM - plan->a_box_rows) * BK * 2;
    const char* rag_env = std::getenv("CCL_GEMM_RAGGED_DENSE");
    const uint32_t rag_bytes = cap > 0 && batch <= kRaggedDense && !(rag_env && atoi(rag_env) == 0) ? (uint32_t)(4 * (kGemmThreads + batch + 1) + 1023) & ~1023u : 0;
    p.rag_dense = rag_bytes ? 1 : 0;
    p.stages = (int32_t)((kSmemBudget - rag_bytes) / p.stage_bytes);
    if (p.stages > 8) p.stages = 8;
    int64_t ntiles = (int64_t)p.tiles_m * p.tiles_n * splits * batch;
    p.batch = (int32_t)batch;
    int units = (int)std::min<int64_t>(ntiles, ctas == 2 ? pairs : sms);
    plan->grid = (unsigned)(units * ctas);
    // grouped raster needs at least one unit per group and whole strips per group
    const bool whole = group_dim == 0 ? p.tiles_n % groups == 0 : group_dim == 1 ? p.tiles_m % groups == 0
                                      : (p.tiles_n % groups_n == 0 && p.tiles_m % (groups / groups_n) == 0);
    if (groups > 1 && units >= groups && whole) {
        p.groups = groups; p.group_dim = group_dim; p.groups_n = groups_n;
    } else { p.groups = 1; p.group_dim = 0; p.groups_n = 1; }
    p.fd_groups_n = make_fastdiv(p.groups_n);
    {   // raster constants (see Scheduler): equal-size groups, floaters, full rounds and the pooled tail
        if (ntiles >= (INT64_C(1) << 31) - 2 * units) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: too many tiles");
        const int gm = p.group_dim == 1 && p.groups > 1 ? p.tiles_m / p.groups : p.group_dim == 2 ? p.tiles_m / (p.groups / p.groups_n) : p.tiles_m;
        const int gn = p.group_dim == 0 && p.groups > 1 ? p.tiles_n / p.groups : p.group_dim == 2 ? p.tiles_n / p.groups_n : p.tiles_n;
        const int64_t per_group = (int64_t)gm * gn * splits * batch;
        p.fd_tiles_per_problem = make_fastdiv((int64_t)gm * gn);
        const int upg = units / p.groups;
        const int64_t rounds = std::min(per_group * p.groups / units, per_group / upg);
        p.sch_units = units; p.sch_gm = gm; p.sch_gn = gn; p.sch_upg = upg; p.sch_floaters = units - upg * p.groups;
        p.sch_rounds = (int32_t)rounds; p.sch_per_group = (int32_t)per_group; p.sch_pool_per_group = (int32_t)(per_group - rounds * upg);
    }
    if (balanced) {                                      // balanced split of the tiles that do not fill a round (see Scheduler)
        units = ctas == 2 ? pairs : sms;
        units -= units % p.groups;
        const int upg = units / p.groups;
        const int64_t rest = p.sch_per_group % upg, work = rest * p.num_kb;
        if (rest > 0) {
            const int64_t sharers = std::max<int64_t>(1, std::min<int64_t>(upg, work / 4));
            plan->grid = (unsigned)(units * ctas);
            p.bal = 1; p.bal_units = (int32_t)sharers; p.bal_tiles = (int32_t)rest;
            p.bal_q = (int32_t)(work / sharers); p.bal_r = (int32_t)(work % sharers);
            p.sch_units = units; p.sch_upg = upg; p.sch_floaters = 0; p.sch_rounds = (int32_t)(p.sch_per_group / upg); p.sch_pool_per_group = 0;
            plan->ws_bytes = (size_t)plan->grid * 2 * ((size_t)BM * bn * 4 + 32);   // two slots of partial sums per CTA, then a flag per slot and epilogue warp
        }
    }
    if (ks) {                                            // cluster split: one cluster per tile, every CTA a part of K
        p.ks = ks; p.kb_per_split = (int32_t)((num_kb + ks - 1) / ks);
        plan->grid = (unsigned)(ntiles * ks);
        p.sch_units = (int32_t)ntiles;
    }
    plan->ks = ks;
    p.fd_num_kb = make_fastdiv(p.num_kb);
    // Raster panel height: the units of a group that run at the same time cover `panel` m-tiles by
    // ceil(upg / panel) n-tiles; all groups walk the same m-panel.  The operand rows + columns such a wave
    // touches are what it pulls from DRAM (the L2 does not hold a wave's footprint until the next wave), so
    // pick the panel that minimises them; ties go to the taller panel.
    {
        const int upg = std::max(1, units / p.groups);
        const int gm = p.sch_gm;
        int64_t best_fp = -1;
        for (int pnl = 1; pnl <= std::min(gm, 64); ++pnl) {
            int64_t fp = (int64_t)pnl * bm + (int64_t)p.groups * ((upg + pnl - 1) / pnl) * bn;
            if (p.group_dim == 1 && p.groups > 1) fp = (int64_t)p.groups * pnl * bm + (int64_t)((upg + pnl - 1) / pnl) * bn;
            if (p.group_dim == 2) fp = (int64_t)(p.groups / p.groups_n) * pnl * bm + (int64_t)p.groups_n * ((upg + pnl - 1) / pnl) * bn;
            if (best_fp < 0 || fp <= best_fp) { best_fp = fp; p.panel = pnl; }
        }
    }
    p.fd_upg = make_fastdiv(p.sch_upg); p.fd_groups = make_fastdiv(p.groups); p.fd_splits = make_fastdiv(p.splits);
    p.fd_per_panel = make_fastdiv((int64_t)p.panel * p.sch_gn); p.fd_panel = make_fastdiv(p.panel);
    p.fd_tps_m = make_fastdiv(p.tps_m); p.fd_tps_n = make_fastdiv(p.tps_n);
    plan->smem_bytes = (uint32_t)p.stages * p.stage_bytes + kEpiBytes + 1024 + (2 * p.stages + 8) * 8 + 16 + rag_bytes;
    p.fd_tiles_n = make_fastdiv(p.tiles_n);
    return CCL_OK;
}

// Rank-5 tensor map of an operand (four coordinates as to_coords() produces them, then the problem of a batch), for
// boxes of box_inner contiguous elements by box_rows strip rows:
//   strips one after the other : {strip row extent, rows per strip, strips, 1}
//   interleaved, mode 1        : {strip row extent, rows per chunk kr, strips, chunk index}; a box of more than kr
//                                rows takes kr rows from each of box_rows / kr consecutive chunks of its strip
//   interleaved, mode 2        : {chunk extent, chunks per strip row, rows per strip, strips}
//   last_strip: of an operand whose last strip is narrower / lower than the others, the map of that strip alone (the
//                map of the others leaves it out)
static ccl_status operand_tmap(CUtensorMap* m, const MatView& v, const void* base, uint32_t box_inner, uint32_t box_rows, int64_t batch, int64_t batch_stride_bytes,
                               bool last_strip = false) {
    uint64_t row = (uint64_t)(v.split == 2 ? v.w : v.cols);      // elements of a strip row
    uint64_t R = (uint64_t)(v.split == 1 ? v.h : v.rows);        // rows per strip
    uint64_t S = (uint64_t)v.nstrips;
    const uint64_t sc = (uint64_t)v.ichunk;
    if (ragged(v)) {
        if (last_strip) {
            base = static_cast<const unsigned char*>(base) + (size_t)(v.nstrips - 1) * (size_t)v.stride * 2;
            if (v.split == 2) row = (uint64_t)v.wlast; else R = (uint64_t)v.hlast;
            S = 1;
        } else S -= 1;
    }
    uint64_t dims[5], strides[4];
    uint32_t box[5];
    int64_t kr;
    const int mode = interleave_mode(v, &kr);
    // last dimension: the problems of a batch (a single entry when the operand is not batched)
    dims[4] = batch > 1 && batch_stride_bytes ? (uint64_t)batch : 1; box[4] = 1;
    if (mode == 1) {
        const uint64_t k = (uint64_t)kr;
        dims[0] = row; dims[1] = k; dims[2] = S; dims[3] = (R + k - 1) / k;
        strides[0] = row * 2; strides[1] = sc * 2; strides[2] = S * sc * 2;
        if (box_rows <= k) { if (k % box_rows) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: a %u-row box does not divide a chunk of %llu rows", box_rows, (unsigned long long)k); }
        else if (box_rows % k) return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: a %u-row box is not made of whole chunks of %llu rows", box_rows, (unsigned long long)k);
        box[0] = box_inner; box[2] = 1;
        if (box_rows <= k) { box[1] = box_rows; box[3] = 1; } else { box[1] = (uint32_t)k; box[3] = box_rows / (uint32_t)k; }
    } else if (mode == 2) {
        dims[0] = sc; dims[1] = row / sc; dims[2] = R; dims[3] = S;
        strides[0] = S * sc * 2; strides[1] = row * S * 2; strides[2] = sc * 2;
        box[0] = box_inner; box[1] = 1; box[2] = box_rows; box[3] = 1;
    } else if (mode == 3) {                              // the buffer as 128-byte lines, fetched one row of a tile at a time
        dims[0] = 64; dims[1] = (uint64_t)(buffer_elems(v) / 64); dims[2] = 1; dims[3] = 1; dims[4] = 1;
        strides[0] = 128; strides[1] = 128; strides[2] = 128;
        box[0] = 64; box[1] = 1; box[2] = 1; box[3] = 1;
    } else if (mode == 0) {
        dims[0] = row; dims[1] = R; dims[2] = v.split ? S : 1; dims[3] = 1;
        strides[0] = row * 2; strides[1] = v.split ? (uint64_t)v.stride * 2 : row * 2; strides[2] = strides[1];
        // (the last strip alone: one strip, so the strip stride is never applied; keep it a multiple of 16 bytes)
        box[0] = box_inner; box[1] = box_rows; box[2] = 1; box[3] = 1;
    } else return fail(CCL_ERR_UNSUPPORTED, "ccl_gemm: this page-interleaved layout has no tensor map");
    strides[3] = dims[4] > 1 ? (uint64_t)batch_stride_bytes : strides[0];
    return encode_tmap(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

}  // namespace ccl

#endif  // CCL_GEMM_PLAN_CUH_
