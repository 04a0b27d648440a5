// Host side of the C ABI declared in include/san.h: argument checks, the arena and
// workspace layout, launch geometry.  Every step of the path runs in the kernels of
// san_kernels.cuh; nothing here computes attention.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <functional>
#include <queue>
#include <vector>
#include <new>

#include "san_ctx.h"
#include "san_kernels.cuh"
#include "san_fused.cuh"
#include "san_step.cuh"
#include "san_rows.cuh"
#include "san_reorder.cuh"
#include "san_learn.cuh"
#include "san_full.cuh"
#include "san_full_tc5.cuh"

using namespace san;

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

int32_t check_config(const san_config* c) {
    if (!c) return SAN_ERR_NULL;
    if (c->n_layers < 1 || c->n_layers > SAN_MAX_LAYERS) return SAN_ERR_SHAPE;
    if (c->n_heads < 1 || c->n_heads > 1024) return SAN_ERR_SHAPE;
    if (c->d_head != kDh) return SAN_ERR_UNSUPPORTED;
    if (c->max_sent < 1 || c->beam < 1 || c->beam > SAN_MAX_BEAM) return SAN_ERR_SHAPE;
    if (c->max_tgt_len < 1 || c->max_src_len < 1) return SAN_ERR_SHAPE;
    if (c->max_tgt_len > (1 << 20) || c->max_src_len > (1 << 20)) return SAN_ERR_SHAPE;
    if ((int64_t)c->max_sent * c->beam > (1 << 24)) return SAN_ERR_SHAPE;
    if (c->dtype != SAN_F32 && c->dtype != SAN_BF16) return SAN_ERR_DTYPE;
    return SAN_OK;
}

// Arena and workspace layout; the one place that knows it.
void layout(const san_config& c, int n_self_planes, int n_enc_planes, san_ctx* L) {
    const size_t e = c.dtype == SAN_F32 ? 4 : 2;
    const size_t n_seqs = (size_t)c.max_sent * c.beam;
    L->elem_bytes = (int)e;
    L->n_seqs = (int)n_seqs;
    L->self_plane_bytes = align_up(n_seqs * c.n_heads * c.max_tgt_len * kDh * e, 256);
    L->mem_plane_bytes = align_up((size_t)c.max_sent * c.n_heads * c.max_src_len * kDh * e, 256);
    L->aan_plane_bytes = align_up(n_seqs * c.n_heads * kDh * sizeof(float), 256);
    L->n_self_k_planes = c.self_is_aan ? 0 : n_self_planes;
    L->n_self_v_planes = c.self_is_aan ? 0 : c.n_layers;
    L->n_enc_k_planes = n_enc_planes;
    L->n_enc_v_planes = c.encdec_shared_context ? n_enc_planes : c.n_layers;
    size_t off = 0;
    L->off_self_k = off; off += L->self_plane_bytes * L->n_self_k_planes;
    L->off_self_v = off; off += L->self_plane_bytes * L->n_self_v_planes;
    L->off_mem_k = off;  off += L->mem_plane_bytes * L->n_enc_k_planes;
    L->off_mem_v = off;  off += L->mem_plane_bytes * L->n_enc_v_planes;
    L->off_aan = off;    off += c.self_is_aan ? L->aan_plane_bytes * c.n_layers : 0;
    L->cache_bytes_needed = std::max<size_t>(off, 256);

    // workspace: error words | tickets [layer][row] | partial sums of split rows
    const size_t rows = n_seqs * c.n_heads;
    L->n_tickets = (size_t)2 * c.n_layers * rows;   // self rows and enc-dec rows of one fused step
    const size_t worst = L->n_tickets * 8 * kDh;   // eight spans per (layer, row), one query row each
    L->part_floats = std::min<size_t>(std::max<size_t>(worst, (size_t)1 << 18), (size_t)1 << 26);
    L->ws_off_tickets = 256;
    L->ws_off_part = align_up(256 + L->n_tickets * sizeof(int), 256);
    L->ws_bytes_needed = L->ws_off_part + L->part_floats * sizeof(float);
}

inline int32_t cuda_status(cudaError_t e) { return e == cudaSuccess ? SAN_OK : SAN_ERR_CUDA; }

constexpr int kQueryGroup = 8;      // query rows (beams) that share a key tile in one work item
int pick_nq_template(int nq) { return nq <= 1 ? 1 : nq <= 2 ? 2 : nq <= 4 ? 4 : 8; }

// Multiplier and shift for FastDiv (exact for dividends below 2^31).
FastDiv make_fastdiv(unsigned d) {
    FastDiv f;
    unsigned shift = 0;
    while ((1ull << shift) < d) ++shift;
    f.shift = shift;
    f.mul = (unsigned)((((unsigned long long)1 << 32) * (((unsigned long long)1 << shift) - d)) / d + 1);
    f.div = d;
    return f;
}
inline int part_header_floats(int nq_t) { return (2 * nq_t + 3) / 4 * 4; }   // (max, sum) per query, 16-byte padded

// Positions per warp item.  Start with one span per row; halve it while the launch would
// leave SMs idle; grow it back if the partial sums would not fit the workspace.
void pick_spans(const san_ctx* ctx, long long units, int max_len, long long part_per_span_floats,
                int* span_len, int* n_spans) {
    const long long target = (long long)ctx->sm_count * 16;
    int sl = (int)align_up((size_t)max_len, 32), ns = 1;
    while (units * ns < target && sl > 32) {
        sl = (int)align_up((size_t)ceil_div(sl, 2), 32);
        ns = ceil_div(max_len, sl);
    }
    while (ns > 1 && part_per_span_floats * ns > (long long)ctx->part_floats) {
        sl = (int)align_up((size_t)sl * 2, 32);
        ns = ceil_div(max_len, sl);
    }
    *span_len = sl;
    *n_spans = ns;
}

// Estimated length of a step of the one-launch kernel for one way of cutting the rows, in
// tiles: a CTA's share of the item list (encoder-memory items first, as in the list) handed to
// its warps greedily, each item to the warp that is free first; the step is as long as the
// busiest warp.  Every row is taken at the host's length bound.
struct CutShape { long long rows; int bound, pi, nq, span, lg; };
double step_makespan(const CutShape& enc, const CutShape& self, int ctas, int tile_rows) {
    constexpr double kItemCost = 1.0;            // tiles' worth of work per item that is not tile arithmetic
    constexpr double kSplitCost = 2.0;           // per span of a split row: partial sums out, ticket, share of the combine
    const int QR = tile_rows - 8;
    auto cost_and_count = [&](const CutShape& c, double* cost, long long* per_cta) {
        if (c.rows == 0) { *cost = 0.0; *per_cta = 0; return; }
        const int ns = ceil_div(c.bound, c.span), nlg = ceil_div(c.pi, c.lg);
        const int span = std::min(c.span, c.bound);
        const int k_tiles = span <= QR ? 1 : 1 + ceil_div(span - QR, tile_rows);
        *cost = k_tiles + (double)c.lg * ceil_div(span, tile_rows) + kItemCost +
                (ns > 1 ? kSplitCost * (1.0 + c.lg * c.nq / 4.0) : 0.0);
        *per_cta = (c.rows * nlg * ns + ctas - 1) / ctas;
    };
    double cost[2]; long long count[2];
    cost_and_count(enc, &cost[0], &count[0]);
    cost_and_count(self, &cost[1], &count[1]);
    std::priority_queue<double, std::vector<double>, std::greater<double>> warps;
    for (int w = 0; w < kFusedWarps; ++w) warps.push(0.0);
    double longest = 0.0;
    for (int k = 0; k < 2; ++k)
        for (long long i = 0; i < count[k]; ++i) {
            const double t = warps.top() + cost[k];
            warps.pop();
            warps.push(t);
            longest = std::max(longest, t);
        }
    return longest;
}

template <typename T>
cudaError_t launch_weights(const WeightsParams& p, int nq_t, unsigned grid, cudaStream_t st) {
    const unsigned block = kWarpsPerCta * 32;
    switch (nq_t) {
        case 1: weights_kernel<T, 1><<<grid, block, 0, st>>>(p); break;
        case 2: weights_kernel<T, 2><<<grid, block, 0, st>>>(p); break;
        case 4: weights_kernel<T, 4><<<grid, block, 0, st>>>(p); break;
        default: weights_kernel<T, 8><<<grid, block, 0, st>>>(p); break;
    }
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_apply(const ApplyParams& p, int nq_t, unsigned grid, cudaStream_t st) {
    const unsigned block = kWarpsPerCta * 32;
    switch (nq_t) {
        case 1: apply_kernel<T, 1><<<grid, block, 0, st>>>(p); break;
        case 2: apply_kernel<T, 2><<<grid, block, 0, st>>>(p); break;
        case 4: apply_kernel<T, 4><<<grid, block, 0, st>>>(p); break;
        default: apply_kernel<T, 8><<<grid, block, 0, st>>>(p); break;
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// The team-pipeline step kernel (san_step.cuh): how the rows are cut into units and how its
// shared memory is laid out.  Returns SAN_ERR_UNSUPPORTED when the shape does not fit (the
// caller then uses the per-warp kernel).
constexpr size_t kStepSmemTotal = 232448;      // opt-in shared memory per CTA on sm_100

struct TeamCut { int spr_log2, lg, tile_pos, zq, rpu; };

int32_t launch_team_step(san_ctx* ctx, const san_step_args* a, int max_len, int max_src, cudaStream_t st, int* rows_per_unit,
                         bool only_if_split, int q_first, int q_count) {
    const san_config& c = ctx->cfg;
    if (c.dtype != SAN_BF16) return SAN_ERR_UNSUPPORTED;
    const bool aan = c.self_is_aan != 0;
    const int n_seqs = a->n_seqs, n_sent = a->n_sent;
    const bool do_self = n_seqs > 0 && !aan, do_enc = n_sent > 0, do_aan = aan && n_seqs > 0;
    const int nqe = pick_nq_template(q_count);
    const int H = c.n_heads;
    int pi_self = 1, pi_enc = 1;
    for (int b = 0; b < ctx->self_pol.n_blocks; ++b) pi_self = std::max(pi_self, ctx->self_pol.size_of_block[b]);
    for (int b = 0; b < ctx->enc_pol.n_blocks; ++b) pi_enc = std::max(pi_enc, ctx->enc_pol.size_of_block[b]);
    if (c.encdec_shared_context) pi_enc = 1;
    const long long rows_self = do_self ? (long long)ctx->self_pol.n_blocks * n_seqs * H : 0;
    const long long rows_enc = do_enc ? (long long)ctx->enc_pol.n_blocks * n_sent * H : 0;
    if (rows_self + rows_enc >= (1ll << 27)) return SAN_ERR_UNSUPPORTED;

    // Long rows are cut into spans handled by the warps of a team (nothing is read twice); short
    // rows are gathered, up to four heads of one sequence or sentence to a warp, so that the cost
    // of a unit beside its arithmetic is shared.  A block's layers go to several units where a
    // unit would otherwise be too fat for the SMs to finish together (each group reads the
    // block's keys again, mostly from L2).
    constexpr int kZCapFloats = 1024;              // score slots a warp may hold per head
    constexpr int kMaxSprLog2 = 1;                 // a row's spans are the warps of one team
    const int rpu_max = H % 4 == 0 ? 4 : H % 2 == 0 ? 2 : 1;
    auto span_of = [](int bound, int spr_log2) { return (int)align_up((size_t)ceil_div(bound, 1 << spr_log2), 16); };
    // What a team's share of the step's bytes is (by the bounds): a unit much fatter than that keeps one
    // team busy after the others have finished, however the units are dealt.
    const double team_share = ((double)rows_self * max_len * (1 + pi_self) + (double)rows_enc * max_src * (1 + pi_enc)) * 128.0 /
                              ((double)ctx->sm_count * kTeams);
    auto cut = [&](long long rows, int bound, int pi, int nq_t, TeamCut* out) -> bool {
        int s = 0, lg = pi;
        while (s < kMaxSprLog2 && span_of(bound, s) * nq_t > kZCapFloats) ++s;
        if (span_of(bound, s) * nq_t > kZCapFloats) return false;
        // Rows of more than 128 positions go to both warps of a team, however many rows there are
        // (measured on 256-position rows: 118.5 us against 128.3 with one warp per row).
        if (s < kMaxSprLog2 && span_of(bound, s) > 128) ++s;
        const int span = span_of(bound, s);
        out->spr_log2 = s;
        out->rpu = s == 0 ? (nq_t > 1 ? std::min(rpu_max, 2) : rpu_max) : 1;   // several queries per head: at most two heads side by side
        out->zq = span + 4;                         // + 4: the score rows of neighbouring queries start in different banks
        // A block's layers go to several units (each of which reads the keys again and recomputes S)
        // only where one unit would otherwise be more than half of a team's share of the whole step:
        // the fat units come first in the list and the small ones fill in behind them.  Measured on
        // 512-position encoder rows of 12 layers beside 256-position self-attention rows: 115.8 us
        // uncut, 118.5 in groups of 6, 122.3 of 4, 127.2 of 3, 136.6 of 2.
        while (lg > 2 && (double)out->rpu * span * 128.0 * (1 + lg) > 0.5 * team_share) lg = std::max(2, ceil_div(lg, 2));
        out->lg = lg;
        // A lone head's span goes through the ring in tiles: 64 positions, so that three slots (of both
        // units of a bundle) fit a team's ring and the producer stays ahead of the consumers.  Several
        // heads side by side need their whole span in one tile.
        out->tile_pos = out->rpu == 1 ? std::min(span, 64) : span;
        return true;
    };
    TeamCut cs{0, 1, 16, 20, 1}, ce{0, 1, 16, 20, 1};
    if (do_self && !cut(rows_self, max_len, pi_self, 1, &cs)) return SAN_ERR_UNSUPPORTED;
    if (do_enc && !cut(rows_enc, max_src, pi_enc, nqe, &ce)) return SAN_ERR_UNSUPPORTED;
    if (ctx->team_cut_override[0] >= 0) {           // testing and tuning: san_step_kernel_select
        // each value may carry a second one for encoder-decoder attention in its bits 8 and up (absent: the same)
        auto pick = [](int v, bool enc) { return enc && (v >> 8) > 0 ? (v >> 8) - 1 : (v & 255); };
        auto apply = [&](TeamCut& tc, bool enc, int bound, int pi, int nq_t) -> bool {
            tc.spr_log2 = std::min(kMaxSprLog2, pick(ctx->team_cut_override[0], enc));
            const int span = span_of(bound, tc.spr_log2);
            if (span * nq_t > kZCapFloats) return false;
            tc.tile_pos = std::min(span, std::max(16, pick(ctx->team_cut_override[2], enc)));
            tc.zq = span + 4;
            int hpu = std::min(rpu_max, std::max(1, pick(ctx->team_cut_override[1], enc)));
            if (hpu == 3) hpu = 2;
            tc.rpu = tc.spr_log2 == 0 ? hpu : 1;
            if (nq_t > 1) tc.rpu = std::min(tc.rpu, 2);
            const int lg = pick(ctx->team_cut_override[3], enc);
            if (lg > 0) tc.lg = std::min(pi, lg);
            return true;
        };
        if (!apply(cs, false, max_len, pi_self, 1) || !apply(ce, true, max_src, pi_enc, nqe)) return SAN_ERR_UNSUPPORTED;
    }

    // Measured on B200 (bench.py, all five workloads): where no row is long enough to be split over
    // the warps of a team, the per-warp kernel is as fast or faster (its 16 warps per SM each
    // carry one row; here 8 consumer warps carry up to four), so the automatic choice keeps
    // this kernel for steps with split rows.
    if (only_if_split && !((do_self && cs.spr_log2 > 0) || (do_enc && ce.spr_log2 > 0))) return SAN_ERR_UNSUPPORTED;

    TeamParams p;
    std::memset(&p, 0, sizeof(p));
    // Shared memory: [ring | pad] per team, then per consumer warp its score slots and its scratch
    // rows (queries, this step's key and value rows), the exchange area of split rows, descriptors,
    // barriers, a row of zeros.  Units of several heads need their whole span in one tile and the
    // tile of every unit of a bundle in the ring: where that does not fit, fewer heads go to a unit;
    // a lone head is cut into tiles of 32 positions.
    size_t zs_bytes = 0, scr_bytes = 0, xo_bytes = 0;
    const bool split = (do_self && cs.spr_log2 > 0) || (do_enc && ce.spr_log2 > 0);
    const int nq_x = std::max(do_self && cs.spr_log2 > 0 ? 1 : 0, do_enc && ce.spr_log2 > 0 ? nqe : 0);
    p.xo_unit_floats = split ? (unsigned)(nq_x * kDh) : 0u;
    xo_bytes = (size_t)kTeams * team_xch_bytes(p.xo_unit_floats);
    for (;;) {
        zs_bytes = align_up((size_t)4 * std::max(do_self ? cs.rpu * cs.zq : 0, do_enc ? ce.rpu * ce.zq * nqe : 0), 16);
        scr_bytes = (size_t)128 * std::max(do_self ? cs.rpu * (2 + cs.lg) : 0, do_enc ? ce.rpu * nqe : 0);
        const size_t tail = kStepConsumers * (zs_bytes + scr_bytes) + xo_bytes + kTeams * kTeamDescBytes + (kTeams * kTeamBarBytes + 16) + 128 + 256;
        if (tail + kTeams * (8 * 1024 + kRingPad) > kStepSmemTotal) return SAN_ERR_UNSUPPORTED;
        p.ring_bytes = (unsigned)(((kStepSmemTotal - tail) / kTeams - kRingPad) / 128 * 128);
        const size_t slot_self = do_self ? (size_t)kTeamWarps * cs.rpu * std::min(cs.tile_pos, max_len) * 128 : 0;   // no row is longer than its bound
        const size_t slot_enc = do_enc ? (size_t)kTeamWarps * ce.rpu * std::min(ce.tile_pos, max_src) * 128 : 0;
        if (slot_self <= p.ring_bytes && slot_enc <= p.ring_bytes) break;
        TeamCut& big = slot_self >= slot_enc ? cs : ce;
        if (big.rpu > 1) big.rpu /= 2;
        else if (big.tile_pos > 64) big.tile_pos = 64;
        else if (big.tile_pos > 32) big.tile_pos = 32;
        else return SAN_ERR_UNSUPPORTED;
    }
    if (rows_per_unit) { rows_per_unit[0] = do_self ? cs.rpu : 0; rows_per_unit[1] = do_enc ? ce.rpu : 0; }
    p.ring_stride = p.ring_bytes + kRingPad;
    p.zs_bytes = (unsigned)zs_bytes; p.scr_bytes = (unsigned)scr_bytes;
    p.off_zs = kTeams * p.ring_stride;
    p.off_scr = (unsigned)(p.off_zs + kStepConsumers * zs_bytes);
    p.off_xo = (unsigned)align_up(p.off_scr + kStepConsumers * scr_bytes, 16);
    p.off_desc = (unsigned)align_up(p.off_xo + xo_bytes, 16);
    p.off_bars = (unsigned)align_up(p.off_desc + kTeams * kTeamDescBytes, 8);
    p.off_zero = (unsigned)align_up(p.off_bars + kTeams * kTeamBarBytes + 16, 128);
    const size_t smem = p.off_zero + 128;

    p.H = H;
    p.err = ctx->err; p.queue = ctx->err + 16;
    p.scale_log2e = (float)(1.4426950408889634 / std::sqrt((double)kDh));
    auto fill = [&](TeamKind& k, const Policy& pol, const TeamCut& tc, int n_it, long long rows, int pi) {
        k.spr_log2 = (unsigned)tc.spr_log2; k.lg_size = (unsigned)tc.lg; k.tile_pos = (unsigned)tc.tile_pos; k.zq = (unsigned)tc.zq;
        k.rpu = (unsigned)tc.rpu;
        const int n_lg = ceil_div(pi, tc.lg);
        k.n_rowlg = (unsigned)(rows / tc.rpu * n_lg);
        k.n_units = (unsigned)align_up((size_t)k.n_rowlg << tc.spr_log2, kTeamWarps);
        k.div_lg = make_fastdiv((unsigned)n_lg); k.div_rows = make_fastdiv((unsigned)std::max(1, n_it * H / tc.rpu)); k.div_h = make_fastdiv((unsigned)H);
        k.n_it = (unsigned)std::max(n_it, 1);
        for (int b = 0; b < pol.n_blocks; ++b) {
            k.first[b] = (unsigned char)pol.first_layer_of_block[b];
            k.size[b] = (unsigned char)pol.size_of_block[b];
        }
    };
    {   // decoder self-attention
        TeamKind& k = p.k[0];
        k.q = static_cast<const char*>(a->d_q_self); k.knew = static_cast<const char*>(a->d_k_new);
        k.vnew = static_cast<const char*>(a->d_v_new);
        k.K = ctx->cache + ctx->off_self_k; k.V = ctx->cache + ctx->off_self_v;
        k.S = a->d_S_self; k.O = static_cast<char*>(a->d_O_self); k.ids = a->d_seq_ids; k.lens = a->d_pos;
        k.plane_bytes = (long long)ctx->self_plane_bytes;
        k.layer_bytes = (long long)n_seqs * H * 128;
        k.S_ld = a->ld_t;
        k.panel_bytes = (unsigned)c.max_tgt_len * 128u;
        k.nq = 1; k.len_bias = 1; k.max_ids = (unsigned)ctx->n_seqs; k.bound = (unsigned)max_len;
        k.q_first = 0; k.q_stride_items = 1; k.v_by_block = 0;
        fill(k, ctx->self_pol, cs, n_seqs, rows_self, pi_self);
    }
    {   // encoder-decoder attention
        TeamKind& k = p.k[1];
        k.q = static_cast<const char*>(a->d_q_enc);
        k.K = ctx->cache + ctx->off_mem_k; k.V = ctx->cache + ctx->off_mem_v;
        k.S = a->d_S_enc; k.O = static_cast<char*>(a->d_O_enc); k.ids = a->d_sent_ids; k.lens = a->d_src_lens;
        k.plane_bytes = (long long)ctx->mem_plane_bytes;
        k.layer_bytes = (long long)n_sent * c.beam * H * 128;
        k.S_ld = a->ld_s;
        k.panel_bytes = (unsigned)c.max_src_len * 128u;
        k.nq = (unsigned)q_count; k.len_bias = 0; k.max_ids = (unsigned)c.max_sent; k.bound = (unsigned)max_src;
        k.q_first = (unsigned)q_first; k.q_stride_items = (unsigned)c.beam; k.v_by_block = c.encdec_shared_context ? 1 : 0;
        fill(k, ctx->enc_pol, ce, n_sent, rows_enc, pi_enc);
    }
    if (!do_self) p.k[0].n_units = 0;
    if (!do_enc) p.k[1].n_units = 0;
    if (do_aan) {
        const int d = H * kDh;
        p.x_aan = static_cast<const char*>(a->d_x_aan); p.t_aan = a->d_t; p.aan_ids = a->d_seq_ids;
        p.aan_sum = reinterpret_cast<float*>(ctx->cache + ctx->off_aan); p.aan_out = static_cast<char*>(a->d_O_self);
        p.n_aan_layers = c.n_layers; p.n_aan_seqs = n_seqs; p.aan_max_seqs = ctx->n_seqs; p.aan_max_t = c.max_tgt_len;
        p.aan_chunks_per_row = ceil_div(d, kAanChunk);
        p.div_aan_chunks = make_fastdiv((unsigned)p.aan_chunks_per_row); p.div_aan_seqs = make_fastdiv((unsigned)n_seqs);
        p.n_aan_units = (unsigned)align_up((size_t)c.n_layers * n_seqs * p.aan_chunks_per_row, kTeamWarps);
    }
    p.n_enc_units = p.k[1].n_units;
    const long long n_units = (long long)p.n_aan_units + p.n_enc_units + p.k[0].n_units;
    if (n_units > (1ll << 30)) return SAN_ERR_UNSUPPORTED;
    p.n_units = (unsigned)n_units;
    if (p.n_units == 0) return SAN_OK;

    const long long bundles = ((long long)p.n_units + kTeamWarps - 1) / kTeamWarps;
    const long long ctas = std::max<long long>(1, std::min<long long>(ctx->sm_count, (bundles + kTeams - 1) / kTeams));
    p.grab_teams = (unsigned)(ctas * kTeams) * (unsigned)std::max(1, ctx->team_grab_mult);

    const void* fn = nqe == 1 ? (const void*)decode_step_team_kernel<1> : nqe == 2 ? (const void*)decode_step_team_kernel<2>
                   : nqe == 4 ? (const void*)decode_step_team_kernel<4> : (const void*)decode_step_team_kernel<8>;
    if (!ctx->team_attr_set) {
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStepSmemTotal) != cudaSuccess) return SAN_ERR_CUDA;
        ctx->team_attr_set = true;
    }
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas); cfg.blockDim = dim3(kStepWarps * 32);
    cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    void* args[] = {&p};
    return cuda_status(cudaLaunchKernelExC(&cfg, fn, args));
}

}  // namespace

extern "C" {

int32_t san_query_bytes(const san_config* cfg, int32_t n_self_blocks, int32_t n_encdec_blocks,
                        size_t* cache_bytes, size_t* workspace_bytes) {
    int32_t rc = check_config(cfg);
    if (rc != SAN_OK) return rc;
    if (n_self_blocks < 1 || n_self_blocks > cfg->n_layers) return SAN_ERR_POLICY;
    if (n_encdec_blocks < 1 || n_encdec_blocks > cfg->n_layers) return SAN_ERR_POLICY;
    san_ctx tmp;
    layout(*cfg, n_self_blocks, n_encdec_blocks, &tmp);
    if (cache_bytes) *cache_bytes = tmp.cache_bytes_needed;
    if (workspace_bytes) *workspace_bytes = tmp.ws_bytes_needed;
    return SAN_OK;
}

int32_t san_create(const san_config* cfg, const int32_t* self_sizes, int32_t n_self,
                   const int32_t* encdec_sizes, int32_t n_encdec, void* d_cache, size_t cache_bytes,
                   void* d_workspace, size_t workspace_bytes, san_ctx** out) {
    if (!out) return SAN_ERR_NULL;
    *out = nullptr;
    int32_t rc = check_config(cfg);
    if (rc != SAN_OK) return rc;
    if (!self_sizes || !encdec_sizes || !d_cache || !d_workspace) return SAN_ERR_NULL;
    Policy ps, pe;
    if ((rc = policy_from_sizes(self_sizes, n_self, cfg->n_layers, &ps)) != SAN_OK) return rc;
    if ((rc = policy_from_sizes(encdec_sizes, n_encdec, cfg->n_layers, &pe)) != SAN_OK) return rc;
    if (((uintptr_t)d_cache & 255) || ((uintptr_t)d_workspace & 255)) return SAN_ERR_SHAPE;
    san_ctx* ctx = new (std::nothrow) san_ctx;
    if (!ctx) return SAN_ERR_CAPACITY;
    ctx->cfg = *cfg;
    ctx->self_pol = ps;
    ctx->enc_pol = pe;
    layout(*cfg, n_self, n_encdec, ctx);
    if (cache_bytes < ctx->cache_bytes_needed || workspace_bytes < ctx->ws_bytes_needed) {
        delete ctx;
        return SAN_ERR_CAPACITY;
    }
    ctx->cache = static_cast<char*>(d_cache);
    ctx->ws = static_cast<char*>(d_workspace);
    ctx->err = reinterpret_cast<int*>(ctx->ws);
    ctx->tickets = reinterpret_cast<int*>(ctx->ws + ctx->ws_off_tickets);
    ctx->part = reinterpret_cast<float*>(ctx->ws + ctx->ws_off_part);
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, dev);
    // error words and tickets start at zero; tickets return to zero after every launch
    if (e == cudaSuccess) e = cudaMemset(ctx->ws, 0, ctx->ws_off_part);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        delete ctx;
        return SAN_ERR_CUDA;
    }
    *out = ctx;
    return SAN_OK;
}

int32_t san_destroy(san_ctx* ctx) {
    if (!ctx) return SAN_ERR_NULL;
    delete ctx;
    return SAN_OK;
}

int32_t san_policy_set_sizes(san_ctx* ctx, int32_t kind, const int32_t* sizes, int32_t n_blocks) {
    if (!ctx || !sizes) return SAN_ERR_NULL;
    if (kind != SAN_SELF && kind != SAN_ENCDEC) return SAN_ERR_RANGE;
    Policy p;
    int32_t rc = policy_from_sizes(sizes, n_blocks, ctx->cfg.n_layers, &p);
    if (rc != SAN_OK) return rc;
    const int planes = kind == SAN_SELF ? (ctx->cfg.self_is_aan ? ctx->cfg.n_layers : ctx->n_self_k_planes)
                                        : ctx->n_enc_k_planes;
    if (p.n_blocks > planes) return SAN_ERR_CAPACITY;
    (kind == SAN_SELF ? ctx->self_pol : ctx->enc_pol) = p;
    ctx->policy_epoch += 1;
    return SAN_OK;
}

int32_t san_policy_set_map(san_ctx* ctx, int32_t kind, const int32_t* block_of_layer, int32_t n_layers) {
    if (!ctx || !block_of_layer) return SAN_ERR_NULL;
    if (kind != SAN_SELF && kind != SAN_ENCDEC) return SAN_ERR_RANGE;
    if (n_layers != ctx->cfg.n_layers) return SAN_ERR_SHAPE;
    Policy p;
    int32_t rc = policy_from_map(block_of_layer, n_layers, &p);
    if (rc != SAN_OK) return rc;
    return san_policy_set_sizes(ctx, kind, p.size_of_block, p.n_blocks);
}

int32_t san_policy_get_map(const san_ctx* ctx, int32_t kind, int32_t* block_of_layer,
                           int32_t* first_layer_of_block, int32_t* n_blocks) {
    if (!ctx) return SAN_ERR_NULL;
    if (kind != SAN_SELF && kind != SAN_ENCDEC) return SAN_ERR_RANGE;
    const Policy& p = kind == SAN_SELF ? ctx->self_pol : ctx->enc_pol;
    if (block_of_layer) std::memcpy(block_of_layer, p.block_of_layer, sizeof(int32_t) * p.n_layers);
    if (first_layer_of_block) std::memcpy(first_layer_of_block, p.first_layer_of_block, sizeof(int32_t) * p.n_blocks);
    if (n_blocks) *n_blocks = p.n_blocks;
    return SAN_OK;
}

int32_t san_cache_append(san_ctx* ctx, int32_t kind, int32_t layer_begin, int32_t layer_end,
                         const void* d_k_new, const void* d_v_new, const int32_t* d_ids,
                         const int32_t* d_pos, const int32_t* d_nrows, int32_t n_items,
                         int32_t rows_per_item, void* stream) {
    if (!ctx || !d_v_new || !d_ids) return SAN_ERR_NULL;
    if (kind != SAN_SELF && kind != SAN_ENCDEC) return SAN_ERR_RANGE;
    const san_config& c = ctx->cfg;
    if (kind == SAN_SELF && c.self_is_aan) return SAN_ERR_UNSUPPORTED;
    if (layer_begin < 0 || layer_end > c.n_layers || layer_begin >= layer_end) return SAN_ERR_RANGE;
    const int cap = kind == SAN_SELF ? c.max_tgt_len : c.max_src_len;
    const int max_ids = kind == SAN_SELF ? ctx->n_seqs : c.max_sent;
    if (n_items < 0 || n_items > max_ids) return SAN_ERR_SHAPE;
    if (rows_per_item < 1 || rows_per_item > cap) return SAN_ERR_SHAPE;
    const Policy& pol = kind == SAN_SELF ? ctx->self_pol : ctx->enc_pol;
    const bool v_by_block = (kind == SAN_ENCDEC && c.encdec_shared_context);

    AppendParams p;
    int n_first = 0;
    for (int l = layer_begin; l < layer_end; ++l) {
        const int lr = l - layer_begin;
        const bool first = pol.is_first(l);
        if (v_by_block && !first) return SAN_ERR_RANGE;   // Eq. 5: upper layers of a block keep no memory
        p.v_plane[lr] = (short)(v_by_block ? pol.block_of_layer[l] : l);
        p.k_plane[lr] = (short)(first ? pol.block_of_layer[l] : -1);
        p.k_src[lr] = (short)(first ? n_first : 0);
        n_first += first ? 1 : 0;
    }
    if (n_first > 0 && !d_k_new) return SAN_ERR_NULL;     // a block-first layer needs its keys
    if (n_first == 0 && d_k_new) return SAN_ERR_RANGE;    // keys offered to layers that keep none
    if (n_items == 0) return SAN_OK;

    const size_t plane = kind == SAN_SELF ? ctx->self_plane_bytes : ctx->mem_plane_bytes;
    p.k_new = static_cast<const char*>(d_k_new);
    p.v_new = static_cast<const char*>(d_v_new);
    p.K = ctx->cache + (kind == SAN_SELF ? ctx->off_self_k : ctx->off_mem_k);
    p.V = ctx->cache + (kind == SAN_SELF ? ctx->off_self_v : ctx->off_mem_v);
    p.k_plane_bytes = (long long)plane;
    p.v_plane_bytes = (long long)plane;
    p.ids = d_ids; p.pos = d_pos; p.nrows = d_nrows;
    p.n_items = n_items; p.rows_per_item = rows_per_item; p.H = c.n_heads; p.cap_len = cap;
    p.max_ids = max_ids; p.n_layers = layer_end - layer_begin; p.row_bytes = kDh * ctx->elem_bytes;
    p.err = ctx->err;
    const long long units = 2LL * p.n_layers * n_items * rows_per_item * c.n_heads * (p.row_bytes / 16);
    const long long grid = (units + 255) / 256;
    if (grid > 0x7fffffffLL) return SAN_ERR_SHAPE;
    append_kernel<<<(unsigned)grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(p);
    return cuda_status(cudaGetLastError());
}

int32_t san_attn_weights(san_ctx* ctx, int32_t kind, int32_t block, const void* d_q,
                         const int32_t* d_ids, const int32_t* d_lens, int32_t n_items,
                         int32_t max_len, float* d_S, int64_t ld_s, void* stream) {
    if (!ctx || !d_q || !d_ids || !d_lens || !d_S) return SAN_ERR_NULL;
    if (kind != SAN_SELF && kind != SAN_ENCDEC) return SAN_ERR_RANGE;
    const san_config& c = ctx->cfg;
    if (kind == SAN_SELF && c.self_is_aan) return SAN_ERR_UNSUPPORTED;
    const Policy& pol = kind == SAN_SELF ? ctx->self_pol : ctx->enc_pol;
    if (block < 0 || block >= pol.n_blocks) return SAN_ERR_RANGE;
    const int cap = kind == SAN_SELF ? c.max_tgt_len : c.max_src_len;
    const int max_ids = kind == SAN_SELF ? ctx->n_seqs : c.max_sent;
    if (n_items < 0 || n_items > max_ids) return SAN_ERR_SHAPE;
    if (max_len == 0) max_len = cap;
    if (max_len < 1 || max_len > cap) return SAN_ERR_SHAPE;
    if (ld_s < max_len) return SAN_ERR_SHAPE;
    if (n_items == 0) return SAN_OK;

    WeightsParams p;
    const size_t plane = kind == SAN_SELF ? ctx->self_plane_bytes : ctx->mem_plane_bytes;
    p.q = d_q;
    p.K = ctx->cache + (kind == SAN_SELF ? ctx->off_self_k : ctx->off_mem_k) + plane * block;
    p.ids = d_ids; p.lens = d_lens; p.S = d_S; p.ld_s = ld_s;
    p.n_items = n_items; p.H = c.n_heads;
    p.nq_total = kind == SAN_SELF ? 1 : c.beam;
    p.cap_len = cap; p.max_ids = max_ids; p.max_len = max_len;
    const long long rows = (long long)n_items * c.n_heads;
    p.part = ctx->part; p.tickets = ctx->tickets; p.err = ctx->err;
    p.scale_log2e = (float)(1.4426950408889634 / std::sqrt((double)kDh));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // a key tile is scored against at most kQueryGroup query rows at a time: larger beams take
    // one launch per group of beams (the groups after the first find the keys in L2)
    for (p.q0 = 0; p.q0 < p.nq_total; p.q0 += kQueryGroup) {
        p.nq = std::min(kQueryGroup, p.nq_total - p.q0);
        pick_spans(ctx, rows, max_len, rows * p.nq * 2, &p.span_len, &p.n_spans_max);
        const long long warps = rows * p.n_spans_max;
        const long long grid = (warps + kWarpsPerCta - 1) / kWarpsPerCta;
        if (grid > 0x7fffffffLL) return SAN_ERR_SHAPE;
        const int nq_t = pick_nq_template(p.nq);
        cudaError_t e = c.dtype == SAN_BF16 ? launch_weights<__nv_bfloat16>(p, nq_t, (unsigned)grid, st)
                                            : launch_weights<float>(p, nq_t, (unsigned)grid, st);
        if (e != cudaSuccess) return SAN_ERR_CUDA;
    }
    return SAN_OK;
}

int32_t san_attn_apply(san_ctx* ctx, int32_t kind, int32_t block, int32_t layer_begin,
                       int32_t layer_end, const float* d_S, int64_t ld_s, const int32_t* d_ids,
                       const int32_t* d_pos_begin, const int32_t* d_pos_end, int32_t n_items,
                       int32_t max_len, void* d_out, int32_t accumulate, void* stream) {
    if (!ctx || !d_S || !d_ids || !d_pos_end || !d_out) return SAN_ERR_NULL;
    if (kind != SAN_SELF && kind != SAN_ENCDEC) return SAN_ERR_RANGE;
    const san_config& c = ctx->cfg;
    if (kind == SAN_SELF && c.self_is_aan) return SAN_ERR_UNSUPPORTED;
    const Policy& pol = kind == SAN_SELF ? ctx->self_pol : ctx->enc_pol;
    if (block < 0 || block >= pol.n_blocks) return SAN_ERR_RANGE;
    const int first = pol.first_layer_of_block[block], size = pol.size_of_block[block];
    if (layer_begin < first || layer_end > first + size || layer_begin >= layer_end) return SAN_ERR_RANGE;
    const bool v_by_block = (kind == SAN_ENCDEC && c.encdec_shared_context);
    if (v_by_block && (layer_begin != first || layer_end != first + 1)) return SAN_ERR_RANGE;
    const int cap = kind == SAN_SELF ? c.max_tgt_len : c.max_src_len;
    const int max_ids = kind == SAN_SELF ? ctx->n_seqs : c.max_sent;
    if (n_items < 0 || n_items > max_ids) return SAN_ERR_SHAPE;
    if (max_len == 0) max_len = cap;
    if (max_len < 1 || max_len > cap) return SAN_ERR_SHAPE;
    if (ld_s < max_len) return SAN_ERR_SHAPE;
    if (n_items == 0) return SAN_OK;

    ApplyParams p;
    const size_t plane = kind == SAN_SELF ? ctx->self_plane_bytes : ctx->mem_plane_bytes;
    const int v_plane0 = v_by_block ? block : layer_begin;
    p.S = d_S; p.ld_s = ld_s;
    p.V = ctx->cache + (kind == SAN_SELF ? ctx->off_self_v : ctx->off_mem_v) + plane * v_plane0;
    p.plane_elems = (long long)(plane / ctx->elem_bytes);
    p.ids = d_ids; p.pos_begin = d_pos_begin; p.pos_end = d_pos_end; p.out = d_out;
    p.n_items = n_items; p.H = c.n_heads;
    p.nq_total = kind == SAN_SELF ? 1 : c.beam;
    p.cap_len = cap; p.max_ids = max_ids; p.max_len = max_len;
    p.n_layers = layer_end - layer_begin;
    p.accumulate = accumulate ? 1 : 0;
    const long long rows = (long long)n_items * c.n_heads;
    // enough rows to fill the GPU: one warp keeps S on chip for every layer of the call;
    // otherwise give each layer its own warp, then split the positions as well
    p.layers_per_warp = (rows >= (long long)ctx->sm_count * 16) ? p.n_layers : 1;
    const int n_lgroups = ceil_div(p.n_layers, p.layers_per_warp);
    p.part = ctx->part; p.tickets = ctx->tickets; p.err = ctx->err;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (p.q0 = 0; p.q0 < p.nq_total; p.q0 += kQueryGroup) {      // one launch per group of beams, as in san_attn_weights
        p.nq = std::min(kQueryGroup, p.nq_total - p.q0);
        pick_spans(ctx, rows * n_lgroups, max_len, rows * p.n_layers * p.nq * kDh, &p.span_len, &p.n_spans_max);
        const long long warps = rows * n_lgroups * p.n_spans_max;
        const long long grid = (warps + kWarpsPerCta - 1) / kWarpsPerCta;
        if (grid > 0x7fffffffLL) return SAN_ERR_SHAPE;
        const int nq_t = pick_nq_template(p.nq);
        cudaError_t e = c.dtype == SAN_BF16 ? launch_apply<__nv_bfloat16>(p, nq_t, (unsigned)grid, st)
                                            : launch_apply<float>(p, nq_t, (unsigned)grid, st);
        if (e != cudaSuccess) return SAN_ERR_CUDA;
    }
    return SAN_OK;
}

int32_t san_aan_step(san_ctx* ctx, int32_t layer_begin, int32_t layer_end, const void* d_x,
                     const int32_t* d_ids, const int32_t* d_t, int32_t n_items, void* d_out,
                     void* stream) {
    if (!ctx || !d_x || !d_ids || !d_t || !d_out) return SAN_ERR_NULL;
    const san_config& c = ctx->cfg;
    if (!c.self_is_aan) return SAN_ERR_UNSUPPORTED;
    if (layer_begin < 0 || layer_end > c.n_layers || layer_begin >= layer_end) return SAN_ERR_RANGE;
    if (n_items < 0 || n_items > ctx->n_seqs) return SAN_ERR_SHAPE;
    if (n_items == 0) return SAN_OK;
    AanParams p;
    p.x = d_x; p.out = d_out;
    p.sum = reinterpret_cast<float*>(ctx->cache + ctx->off_aan);
    p.ids = d_ids; p.t = d_t; p.n_items = n_items; p.d = c.n_heads * kDh;
    p.max_ids = ctx->n_seqs; p.max_t = c.max_tgt_len;
    p.n_layers = layer_end - layer_begin; p.layer_begin = layer_begin; p.err = ctx->err;
    const long long units = (long long)p.n_layers * n_items * (p.d / 4);
    const long long grid = (units + 255) / 256;
    if (grid > 0x7fffffffLL) return SAN_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (c.dtype == SAN_BF16) aan_kernel<__nv_bfloat16><<<(unsigned)grid, 256, 0, st>>>(p);
    else aan_kernel<float><<<(unsigned)grid, 256, 0, st>>>(p);
    return cuda_status(cudaGetLastError());
}

int32_t san_seq_reset(san_ctx* ctx, const int32_t* d_seq_ids, int32_t n, void* stream) {
    if (!ctx || (n > 0 && !d_seq_ids)) return SAN_ERR_NULL;
    const san_config& c = ctx->cfg;
    if (!c.self_is_aan) return SAN_ERR_UNSUPPORTED;
    if (n < 0 || n > ctx->n_seqs) return SAN_ERR_SHAPE;
    if (n == 0) return SAN_OK;
    ResetParams p;
    p.sum = reinterpret_cast<float*>(ctx->cache + ctx->off_aan);
    p.ids = d_seq_ids; p.n_items = n; p.d = c.n_heads * kDh; p.max_ids = ctx->n_seqs; p.n_layers = c.n_layers;
    p.err = ctx->err;
    const long long units = (long long)p.n_layers * n * (p.d / 4);
    const long long grid = (units + 255) / 256;
    if (grid > 0x7fffffffLL) return SAN_ERR_SHAPE;
    aan_reset_kernel<<<(unsigned)grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(p);
    return cuda_status(cudaGetLastError());
}

// One launch of the step for the query rows (beams) [q_first, q_first + q_count) of every sentence;
// n_seqs > 0 in `a` adds the self-attention (or AAN) part.  Arguments have been checked.
static int32_t decode_step_launch(san_ctx* ctx, const san_step_args* a, int max_len, int max_src, int q_first, int q_count, void* stream) {
    const san_config& c = ctx->cfg;
    const bool aan = c.self_is_aan != 0;
    const int n_seqs = a->n_seqs, n_sent = a->n_sent;
    const bool bf16 = c.dtype == SAN_BF16;
    if (ctx->step_kernel == 0 || ctx->step_kernel == 2) {       // automatic: the team-pipeline kernel for steps with rows long enough to be split over a team
        const int32_t rc = launch_team_step(ctx, a, max_len, max_src, static_cast<cudaStream_t>(stream), ctx->last_rows_per_unit,
                                            ctx->step_kernel == 0 && ctx->team_cut_override[0] < 0, q_first, q_count);
        if (rc != SAN_ERR_UNSUPPORTED) { ctx->last_step_kernel = 2; return rc; }
        if (ctx->step_kernel == 2) return rc;
    }
    ctx->last_step_kernel = 1;
    const int row_bytes = kDh * ctx->elem_bytes;
    const int TR = kStageBytes / row_bytes;
    const int nqe = pick_nq_template(q_count);
    const bool do_self = n_seqs > 0 && !aan;
    const bool do_enc = n_sent > 0;
    // Sentence-sized rows (every row a handful of 16-position blocks): the kernel that takes a whole
    // plane per copy and keeps the scores in registers.  An item is 1, 2 or 4 heads of a (block,
    // sequence): as many as the head count divides by, the warp's ring holds as one plane, and the
    // registers hold the weights of.
    auto rows_heads = [&](int bound, int nq, int want) {
        for (int r = 4; r >= 1; r >>= 1) {
            if (r > want || c.n_heads % r) continue;
            if (r * (bound + nq) > kRowsRingRows || r * nq > 8) continue;
            if (ceil_div(bound, 16) > rows_max_blocks(r)) continue;
            return r;
        }
        return 0;
    };
    int hpi_self = 1, hpi_enc = 1;
    bool use_rows = false;
    // Measured on B200 (sentence-sized workload, microbench/step_kernels.py): a launch with encoder-decoder
    // attention alone takes 9.3 us with this kernel (one head per item) against 19.7 us with the per-warp
    // kernel; with self-attention in the launch the two are level (23.3 against 23.1 us), and beside the
    // running averages the per-warp kernel is ahead (13.4 against 14.3 us).  So automatically it takes the
    // launches without a self-attention part: the query groups of a wide beam after the first.
    const bool rows_auto = ctx->step_kernel == 0 && n_seqs == 0 && do_enc;
    if (bf16 && (ctx->step_kernel == 3 || rows_auto)) {
        const int o = ctx->team_cut_override[1];       // heads per item wanted: as in san_step_kernel_select
        const int want_self = ctx->step_kernel == 3 && (o & 255) > 0 ? (o & 255) : 2;
        const int want_enc = ctx->step_kernel == 3 ? ((o >> 8) > 0 ? (o >> 8) - 1 : (o & 255) > 0 ? (o & 255) : 1) : 1;
        const int rs = do_self ? rows_heads(max_len, 1, want_self) : 1, re = do_enc ? rows_heads(max_src, nqe, want_enc) : 1;
        if (rs > 0 && re > 0) { use_rows = true; hpi_self = rs; hpi_enc = re; }
    }
    if (ctx->step_kernel == 3 && !use_rows) return SAN_ERR_UNSUPPORTED;
    int pi_self = 1, pi_enc = 1;
    for (int b = 0; b < ctx->self_pol.n_blocks; ++b) pi_self = std::max(pi_self, ctx->self_pol.size_of_block[b]);
    for (int b = 0; b < ctx->enc_pol.n_blocks; ++b) pi_enc = std::max(pi_enc, ctx->enc_pol.size_of_block[b]);
    if (c.encdec_shared_context) pi_enc = 1;
    const long long rows_self = do_self ? (long long)ctx->self_pol.n_blocks * n_seqs * (c.n_heads / hpi_self) : 0;
    const long long rows_enc = do_enc ? (long long)ctx->enc_pol.n_blocks * n_sent * (c.n_heads / hpi_enc) : 0;
    if ((size_t)(rows_self + rows_enc) > ctx->n_tickets) return SAN_ERR_CAPACITY;

    // positions per item: what the on-chip score buffer holds, then smaller while items are
    // fat (long tails) or too few to fill the persistent warps
    // Work per item.  An item is one warp's serial chain of tiles (key panel, then the value
    // panels of its layers), so its length bounds both the step time and the balance: keep it
    // to about half of a warp's share of all tiles, never under kMinTiles.  A long chain
    // is first cut by layers: a block's layers go to several items, each of which recomputes
    // the block's S from the keys (extra key reads, nothing to combine; never fewer than two
    // layers per item, or sharing would buy nothing), or by positions: spans of a row whose
    // partial sums the last span to finish combines.  Spans are multiples of 16 rows and
    // at most what the on-chip score buffer holds.
    constexpr long long kMinTiles = 8;
    const int QR = TR - 8;                                           // key rows beside the queries in an item's first tile
    auto tiles_of = [&](int span, int layers) {
        const int k_tiles = span <= QR ? 1 : 1 + ceil_div(span - QR, TR);
        return (long long)k_tiles + (long long)layers * ceil_div(span, TR);
    };
    const long long warps = (long long)ctx->sm_count * kFusedWarps;
    const int cap_self = std::min(kZFloats, (int)align_up((size_t)max_len, 16)), cap_enc = std::min(kZFloats / nqe, (int)align_up((size_t)max_src, 16));
    const long long total_tiles = (do_self ? rows_self * ceil_div(max_len, cap_self) * tiles_of(cap_self, pi_self) : 0) +
                                  (do_enc ? rows_enc * ceil_div(max_src, cap_enc) * tiles_of(cap_enc, pi_enc) : 0);
    const long long budget = std::max<long long>(kMinTiles, total_tiles / (2 * warps));
    auto pick = [&](int cap, int pi, int nq, int* span, int* lg_size) {
        int sp = cap, lg = pi;
        if (nq == 1) {      // one query row: partial sums are small and quick to combine, so cut positions first
            while (sp > 64 && tiles_of(sp, lg) > budget) sp = std::max(64, (int)align_up((size_t)ceil_div(sp, 2), 16));
            while (lg > 2 && tiles_of(sp, lg) > budget) lg = std::max(2, ceil_div(lg, 2));
        } else {            // several query rows share a tile: partial sums are nq times bigger, so cut layers first
            while (lg > 2 && tiles_of(sp, lg) > budget) lg = std::max(2, ceil_div(lg, 2));
            while (sp > 32 && tiles_of(sp, lg) > 2 * budget) sp = std::max(32, (int)align_up((size_t)ceil_div(sp, 2), 16));
        }
        *span = sp; *lg_size = lg;
    };
    int span_self = cap_self, span_enc = cap_enc, lg_self = pi_self, lg_enc = pi_enc;
    pick(cap_self, pi_self, 1, &span_self, &lg_self);
    pick(cap_enc, pi_enc, q_count, &span_enc, &lg_enc);
    // The rule above looks at one item at a time.  Where it cuts anything, compare it with the other
    // ways of cutting (halved spans, halved layer groups, or no cut at all) by the estimated length
    // of the step: items of equal size that divide evenly over the warps beat smaller items that
    // leave a warp with one more than its neighbours.  The choice is remembered per launch shape.
    if (use_rows) {      // whole rows; layers per item as above unless told otherwise
        span_self = cap_self; span_enc = cap_enc;
        const int o = ctx->team_cut_override[3];
        const int o_enc = (o >> 8) > 0 ? (o >> 8) - 1 : (o & 255);     // as in san_step_kernel_select
        if (ctx->step_kernel == 3 && (o & 255) > 0) lg_self = std::min(pi_self, o & 255);
        if (ctx->step_kernel == 3 && o_enc > 0) lg_enc = std::min(pi_enc, o_enc);
    } else if (span_self < cap_self || lg_self < pi_self || span_enc < cap_enc || lg_enc < pi_enc) {
        const int len_b = std::min(c.max_tgt_len, (int)align_up((size_t)max_len, TR)), src_b = std::min(c.max_src_len, (int)align_up((size_t)max_src, TR));
        san_ctx::StepPlan* plan = nullptr;
        for (auto& pl : ctx->plans)
            if (pl.valid && pl.epoch == ctx->policy_epoch && pl.n_seqs == n_seqs && pl.n_sent == n_sent &&
                pl.len_bound == len_b && pl.src_bound == src_b) plan = &pl;
        if (!plan) {
            const int ctas = (int)std::max<long long>(1, std::min<long long>(ctx->sm_count, (rows_self + rows_enc + kFusedWarps - 1) / kFusedWarps));
            CutShape ce{rows_enc, src_b, pi_enc, q_count, span_enc, lg_enc}, cs{rows_self, len_b, pi_self, 1, span_self, lg_self};
            double best = step_makespan(ce, cs, ctas, TR);
            int b_ss = span_self, b_ls = lg_self, b_se = span_enc, b_le = lg_enc;
            auto halvings = [](int from, int floor_, int align, std::vector<int>* out) {
                for (int v = from;; v = std::max(floor_, (int)align_up((size_t)ceil_div(v, 2), align))) {
                    out->push_back(v);
                    if (v <= floor_) break;
                }
            };
            std::vector<int> ss, ls, se, le;
            halvings(cap_self, std::min(cap_self, 64), 16, &ss); halvings(pi_self, std::min(pi_self, 2), 1, &ls);
            halvings(cap_enc, std::min(cap_enc, 32), 16, &se);   halvings(pi_enc, std::min(pi_enc, 2), 1, &le);
            if (!do_self) { ss.assign(1, span_self); ls.assign(1, lg_self); }
            if (!do_enc) { se.assign(1, span_enc); le.assign(1, lg_enc); }
            for (int a : ss) for (int b : ls) for (int d : se) for (int e : le) {
                if (ceil_div(len_b, a) > kMaxSpans || ceil_div(src_b, d) > kMaxSpans) continue;
                const long long need = (ceil_div(len_b, a) > 1 ? rows_self * ceil_div(pi_self, b) * ceil_div(len_b, a) * (part_header_floats(1) + b * kDh) : 0) +
                                       (ceil_div(src_b, d) > 1 ? rows_enc * ceil_div(pi_enc, e) * ceil_div(src_b, d) * (part_header_floats(nqe) + e * nqe * kDh) : 0);
                if (need > (long long)ctx->part_floats) continue;
                cs.span = a; cs.lg = b; ce.span = d; ce.lg = e;
                const double t = step_makespan(ce, cs, ctas, TR);
                if (t < 0.97 * best) { best = t; b_ss = a; b_ls = b; b_se = d; b_le = e; }
            }
            plan = &ctx->plans[ctx->plan_next];
            ctx->plan_next = (ctx->plan_next + 1) % san_ctx::kPlans;
            plan->valid = true; plan->epoch = ctx->policy_epoch; plan->n_seqs = n_seqs; plan->n_sent = n_sent;
            plan->len_bound = len_b; plan->src_bound = src_b;
            plan->span_self = b_ss; plan->lg_self = b_ls; plan->span_enc = b_se; plan->lg_enc = b_le;
        }
        span_self = plan->span_self; lg_self = plan->lg_self; span_enc = plan->span_enc; lg_enc = plan->lg_enc;
    }
    // a row may be cut into at most kMaxSpans spans of at most what the score buffer holds
    if (do_self && ceil_div(max_len, kZFloats) > kMaxSpans) return SAN_ERR_UNSUPPORTED;
    if (do_enc && ceil_div(max_src, kZFloats / nqe) > kMaxSpans) return SAN_ERR_UNSUPPORTED;
    while (do_self && ceil_div(max_len, span_self) > kMaxSpans && span_self < kZFloats) span_self = std::min(kZFloats, span_self * 2);
    while (do_enc && ceil_div(max_src, span_enc) > kMaxSpans && span_enc < kZFloats / nqe) span_enc = std::min(kZFloats / nqe, span_enc * 2);
    const int nlg_self = ceil_div(pi_self, lg_self), nlg_enc = ceil_div(pi_enc, lg_enc);
    const long long rl_self = rows_self * nlg_self, rl_enc = rows_enc * nlg_enc;      // (row, layer group) pairs
    if ((size_t)(rl_self + rl_enc) > ctx->n_tickets) return SAN_ERR_CAPACITY;
    const int stride_self = part_header_floats(1) + lg_self * kDh, stride_enc = part_header_floats(nqe) + lg_enc * nqe * kDh;
    auto part_need = [&]() {
        const int ns = ceil_div(max_len, span_self), ne = ceil_div(max_src, span_enc);
        return (ns > 1 ? rl_self * ns * stride_self : 0) + (ne > 1 ? rl_enc * ne * stride_enc : 0);
    };
    while (part_need() > (long long)ctx->part_floats) {   // fewer, longer spans until the partial sums fit
        if (span_self < kZFloats && ceil_div(max_len, span_self) > 1 &&
            (long long)rl_self * stride_self * ceil_div(max_len, span_self) >= (long long)rl_enc * stride_enc * ceil_div(max_src, span_enc))
            span_self = std::min(kZFloats, span_self * 2);
        else if (span_enc < kZFloats / nqe && ceil_div(max_src, span_enc) > 1) span_enc = std::min(kZFloats / nqe, span_enc * 2);
        else if (span_self < kZFloats && ceil_div(max_len, span_self) > 1) span_self = std::min(kZFloats, span_self * 2);
        else return SAN_ERR_UNSUPPORTED;
    }
    const int ns_self = do_self ? ceil_div(max_len, span_self) : 1, ns_enc = do_enc ? ceil_div(max_src, span_enc) : 1;
    if (ns_self > kMaxSpans || ns_enc > kMaxSpans) return SAN_ERR_UNSUPPORTED;

    if ((long long)ctx->n_seqs * c.n_heads * c.n_layers >= (1ll << 31)) return SAN_ERR_UNSUPPORTED;   // 32-bit row indices
    if (rl_enc * ns_enc + rl_self * ns_self > (1ll << 30)) return SAN_ERR_UNSUPPORTED;
    StepParams p;
    std::memset(&p, 0, sizeof(p));
    p.H = c.n_heads;
    p.n_enc_items = (unsigned)(rl_enc * ns_enc); p.n_items = p.n_enc_items + (unsigned)(rl_self * ns_self);
    p.part = ctx->part; p.tickets = ctx->tickets; p.err = ctx->err;
    p.scale_log2e = (float)(1.4426950408889634 / std::sqrt((double)kDh));
    {   // decoder self-attention
        KindParams& k = p.k[0];
        k.q = static_cast<const char*>(a->d_q_self); k.knew = static_cast<const char*>(a->d_k_new);
        k.vnew = static_cast<const char*>(a->d_v_new);
        k.K = ctx->cache + ctx->off_self_k; k.V = ctx->cache + ctx->off_self_v;
        k.S = a->d_S_self; k.O = static_cast<char*>(a->d_O_self); k.ids = a->d_seq_ids; k.lens = a->d_pos;
        k.plane_bytes = (long long)ctx->self_plane_bytes;
        k.layer_bytes = (long long)n_seqs * c.n_heads * row_bytes;
        k.S_ld = a->ld_t;
        k.part_base = ns_enc > 1 ? rl_enc * ns_enc * stride_enc : 0;
        k.panel_bytes = (unsigned)c.max_tgt_len * row_bytes;
        k.n_it = (unsigned)std::max(n_seqs, 1); k.nq = 1; k.q_first = 0; k.q_total = 1; k.len_bias = 1; k.max_ids = (unsigned)ctx->n_seqs; k.bound = (unsigned)max_len;
        k.span = (unsigned)span_self; k.nspans = (unsigned)ns_self; k.part_stride = (unsigned)stride_self; k.v_by_block = 0;
        k.row_base = (unsigned)rl_enc;
        k.lg_size = (unsigned)lg_self; k.n_lg = (unsigned)nlg_self; k.div_lg = make_fastdiv((unsigned)nlg_self);
        k.hpi = (unsigned)hpi_self;
        k.div_span = make_fastdiv((unsigned)ns_self); k.div_h = make_fastdiv((unsigned)(c.n_heads / hpi_self)); k.div_item = make_fastdiv(k.n_it);
        for (int b = 0; b < ctx->self_pol.n_blocks; ++b) {
            k.first[b] = (unsigned char)ctx->self_pol.first_layer_of_block[b];
            k.size[b] = (unsigned char)ctx->self_pol.size_of_block[b];
        }
    }
    {   // encoder-decoder attention
        KindParams& k = p.k[1];
        k.q = static_cast<const char*>(a->d_q_enc); k.knew = nullptr; k.vnew = nullptr;
        k.K = ctx->cache + ctx->off_mem_k; k.V = ctx->cache + ctx->off_mem_v;
        k.S = a->d_S_enc; k.O = static_cast<char*>(a->d_O_enc); k.ids = a->d_sent_ids; k.lens = a->d_src_lens;
        k.plane_bytes = (long long)ctx->mem_plane_bytes;
        k.layer_bytes = (long long)n_sent * c.beam * c.n_heads * row_bytes;
        k.S_ld = a->ld_s;
        k.part_base = 0;
        k.panel_bytes = (unsigned)c.max_src_len * row_bytes;
        k.n_it = (unsigned)std::max(n_sent, 1); k.nq = (unsigned)q_count; k.q_first = (unsigned)q_first; k.q_total = (unsigned)c.beam; k.len_bias = 0; k.max_ids = (unsigned)c.max_sent; k.bound = (unsigned)max_src;
        k.span = (unsigned)span_enc; k.nspans = (unsigned)ns_enc; k.part_stride = (unsigned)stride_enc;
        k.v_by_block = c.encdec_shared_context ? 1 : 0;
        k.row_base = 0;
        k.lg_size = (unsigned)lg_enc; k.n_lg = (unsigned)nlg_enc; k.div_lg = make_fastdiv((unsigned)nlg_enc);
        k.hpi = (unsigned)hpi_enc;
        k.div_span = make_fastdiv((unsigned)ns_enc); k.div_h = make_fastdiv((unsigned)(c.n_heads / hpi_enc)); k.div_item = make_fastdiv(k.n_it);
        for (int b = 0; b < ctx->enc_pol.n_blocks; ++b) {
            k.first[b] = (unsigned char)ctx->enc_pol.first_layer_of_block[b];
            k.size[b] = (unsigned char)ctx->enc_pol.size_of_block[b];
        }
    }
    if (aan && n_seqs > 0) {
        p.x_aan = static_cast<const char*>(a->d_x_aan); p.t_aan = a->d_t; p.aan_ids = a->d_seq_ids;
        p.aan_sum = reinterpret_cast<float*>(ctx->cache + ctx->off_aan); p.aan_out = static_cast<char*>(a->d_O_self);
        p.n_aan_layers = c.n_layers; p.n_aan_seqs = n_seqs; p.aan_max_seqs = ctx->n_seqs; p.aan_max_t = c.max_tgt_len;
    }

    if (use_rows) {
        ctx->last_step_kernel = 3;
        ctx->last_rows_per_unit[0] = hpi_self; ctx->last_rows_per_unit[1] = hpi_enc;
        const void* rfn = (const void*)decode_step_rows_kernel;
        const size_t rsmem = rows_smem_bytes();
        if (!ctx->rows_attr_set) {
            if (cudaFuncSetAttribute(rfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)rsmem) != cudaSuccess) return SAN_ERR_CUDA;
            ctx->rows_attr_set = true;
        }
        long long rctas = std::min<long long>(ctx->sm_count, p.n_items);      // few items: spread them over the SMs rather than fill the warps of fewer
        if (p.x_aan) rctas = ctx->sm_count;
        if (rctas < 1) rctas = 1;
        cudaLaunchAttribute rattr;
        rattr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        rattr.val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t rcfg = {};
        rcfg.gridDim = dim3((unsigned)rctas); rcfg.blockDim = dim3(kRowsWarps * 32);
        rcfg.dynamicSmemBytes = rsmem; rcfg.stream = static_cast<cudaStream_t>(stream);
        rcfg.attrs = &rattr; rcfg.numAttrs = 1;
        void* rargs[] = {&p};
        return cuda_status(cudaLaunchKernelExC(&rcfg, rfn, rargs));
    }
    const void* fn = nullptr;
    if (bf16) fn = nqe == 1 ? (const void*)decode_step_kernel<__nv_bfloat16, 1> : nqe == 2 ? (const void*)decode_step_kernel<__nv_bfloat16, 2>
                   : nqe == 4 ? (const void*)decode_step_kernel<__nv_bfloat16, 4> : (const void*)decode_step_kernel<__nv_bfloat16, 8>;
    else fn = nqe == 1 ? (const void*)decode_step_kernel<float, 1> : nqe == 2 ? (const void*)decode_step_kernel<float, 2>
              : nqe == 4 ? (const void*)decode_step_kernel<float, 4> : (const void*)decode_step_kernel<float, 8>;
    const size_t smem = fused_smem_bytes();
    if (!ctx->fused_attr_set) {
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return SAN_ERR_CUDA;
        ctx->fused_attr_set = true;
    }
    long long ctas = std::min<long long>(ctx->sm_count, (p.n_items + kFusedWarps - 1) / kFusedWarps);
    if (p.x_aan) ctas = ctx->sm_count;     // the running average is spread over every thread of the grid
    if (ctas < 1) ctas = 1;
    // Programmatic stream serialization: the grid may be scheduled while the preceding kernel of
    // the stream is finishing; the kernel touches no global memory before that kernel is complete.
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas); cfg.blockDim = dim3(kFusedWarps * 32);
    cfg.dynamicSmemBytes = smem; cfg.stream = static_cast<cudaStream_t>(stream);
    cfg.attrs = &attr; cfg.numAttrs = 1;
    void* args[] = {&p};
    cudaError_t e = cudaLaunchKernelExC(&cfg, fn, args);
    return cuda_status(e);
}

int32_t san_decode_step(san_ctx* ctx, const san_step_args* a, void* stream) {
    if (!ctx || !a) return SAN_ERR_NULL;
    const san_config& c = ctx->cfg;
    const bool aan = c.self_is_aan != 0;
    const int n_seqs = a->n_seqs, n_sent = a->n_sent;
    if (n_seqs < 0 || n_seqs > ctx->n_seqs || n_sent < 0 || n_sent > c.max_sent) return SAN_ERR_SHAPE;
    if (n_seqs > 0) {
        if (!a->d_seq_ids || !a->d_O_self) return SAN_ERR_NULL;
        if (aan ? (!a->d_x_aan || !a->d_t) : (!a->d_q_self || !a->d_k_new || !a->d_v_new || !a->d_pos)) return SAN_ERR_NULL;
    }
    if (n_sent > 0 && (!a->d_q_enc || !a->d_sent_ids || !a->d_src_lens || !a->d_O_enc)) return SAN_ERR_NULL;
    int max_len = a->max_len == 0 ? c.max_tgt_len : a->max_len;
    int max_src = a->max_src == 0 ? c.max_src_len : a->max_src;
    if (max_len < 1 || max_len > c.max_tgt_len || max_src < 1 || max_src > c.max_src_len) return SAN_ERR_SHAPE;
    if (n_seqs > 0 && !aan && a->d_S_self && a->ld_t < max_len) return SAN_ERR_SHAPE;
    if (n_sent > 0 && a->d_S_enc && a->ld_s < max_src) return SAN_ERR_SHAPE;
    if (n_seqs == 0 && n_sent == 0) return SAN_OK;

    // A key tile is scored against at most kQueryGroup query rows at a time.  Wider beams take one
    // launch per group of beams: the first also carries the self-attention (or AAN) part, the
    // others read the encoder memory again (mostly from L2).
    san_step_args part = *a;
    for (int q0 = 0; q0 == 0 || (n_sent > 0 && q0 < c.beam); q0 += kQueryGroup) {
        if (q0 > 0) part.n_seqs = 0;
        const int32_t rc = decode_step_launch(ctx, &part, max_len, max_src, q0, std::min(kQueryGroup, c.beam - q0), stream);
        if (rc != SAN_OK) return rc;
    }
    return SAN_OK;
}

int32_t san_step_kernel_select(san_ctx* ctx, int32_t which, int32_t spans_log2, int32_t heads_per_unit, int32_t tile_pos,
                               int32_t layers_per_unit, int32_t grab_mult) {
    if (!ctx) return SAN_ERR_NULL;
    if (which < 0 || which > 3) return SAN_ERR_RANGE;
    // every value may carry a second one for encoder-decoder attention in its bits 8 and up, as (v + 1) << 8
    auto both = [](int32_t v, bool (*ok)(int32_t)) { return v >= 0 && ok(v & 255) && ((v >> 8) == 0 || ((v >> 8) <= 256 && ok((v >> 8) - 1))); };
    if (spans_log2 >= 0 && !both(tile_pos, [](int32_t t) { return t >= 16 && t <= 240 && t % 16 == 0; })) return SAN_ERR_RANGE;
    if (!both(heads_per_unit, [](int32_t h) { return h >= 1 && h <= 4; })) return SAN_ERR_RANGE;
    if (spans_log2 >= 0 && !both(spans_log2, [](int32_t v) { return v <= 1; })) return SAN_ERR_RANGE;
    if (!both(layers_per_unit, [](int32_t v) { return v <= SAN_MAX_LAYERS; })) return SAN_ERR_RANGE;
    ctx->step_kernel = which;
    ctx->team_cut_override[0] = spans_log2 < 0 ? -1 : spans_log2;
    ctx->team_cut_override[1] = heads_per_unit;
    ctx->team_cut_override[2] = tile_pos;
    ctx->team_cut_override[3] = layers_per_unit;
    ctx->team_grab_mult = grab_mult > 0 ? grab_mult : 1;
    return SAN_OK;
}

int32_t san_step_kernel_used(const san_ctx* ctx, int32_t* which, int32_t* rows_per_unit) {
    if (!ctx || !which) return SAN_ERR_NULL;
    *which = ctx->last_step_kernel;
    if (rows_per_unit) { rows_per_unit[0] = ctx->last_step_kernel >= 2 ? ctx->last_rows_per_unit[0] : 0; rows_per_unit[1] = ctx->last_step_kernel >= 2 ? ctx->last_rows_per_unit[1] : 0; }
    return SAN_OK;
}

int32_t san_decode_step_host(san_ctx* ctx, const san_step_args* h, const san_step_args* d, void* stream) {
    if (!ctx || !h || !d) return SAN_ERR_NULL;
    const san_config& c = ctx->cfg;
    const bool aan = c.self_is_aan != 0;
    const int n_seqs = d->n_seqs, n_sent = d->n_sent;
    if (n_seqs < 0 || n_seqs > ctx->n_seqs || n_sent < 0 || n_sent > c.max_sent) return SAN_ERR_SHAPE;
    const size_t row = (size_t)c.n_heads * kDh * ctx->elem_bytes;           // one sequence, all heads
    const size_t Ns = (size_t)ctx->self_pol.n_blocks, Ne = (size_t)ctx->enc_pol.n_blocks, M = (size_t)c.n_layers;
    const size_t n_enc_out = c.encdec_shared_context ? Ne : M;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    struct Copy { const void* from; const void* to; size_t bytes; };
    // inputs: host -> the caller's device buffers
    const Copy in[] = {
        {h->d_seq_ids, d->d_seq_ids, n_seqs * sizeof(int32_t)},
        {aan ? nullptr : h->d_pos, d->d_pos, n_seqs * sizeof(int32_t)},
        {aan ? nullptr : h->d_q_self, d->d_q_self, Ns * n_seqs * row},
        {aan ? nullptr : h->d_k_new, d->d_k_new, Ns * n_seqs * row},
        {aan ? nullptr : h->d_v_new, d->d_v_new, M * n_seqs * row},
        {aan ? h->d_x_aan : nullptr, d->d_x_aan, M * n_seqs * row},
        {aan ? h->d_t : nullptr, d->d_t, n_seqs * sizeof(int32_t)},
        {h->d_sent_ids, d->d_sent_ids, n_sent * sizeof(int32_t)},
        {h->d_src_lens, d->d_src_lens, n_sent * sizeof(int32_t)},
        {h->d_q_enc, d->d_q_enc, Ne * n_sent * c.beam * row},
    };
    for (const Copy& cp : in) {
        if (cp.bytes == 0 || (!cp.from && !cp.to)) continue;
        if (!cp.from || !cp.to) return SAN_ERR_NULL;
    }
    const Copy out[] = {
        {d->d_O_self, h->d_O_self, M * n_seqs * row},
        {d->d_O_enc, h->d_O_enc, n_enc_out * n_sent * c.beam * row},
        {d->d_S_self, h->d_S_self, aan ? 0 : Ns * n_seqs * c.n_heads * (size_t)d->ld_t * sizeof(float)},
        {d->d_S_enc, h->d_S_enc, Ne * n_sent * c.beam * c.n_heads * (size_t)d->ld_s * sizeof(float)},
    };
    for (int i = 0; i < 2; ++i)
        if (out[i].bytes && (!out[i].from || !out[i].to)) return SAN_ERR_NULL;
    for (const Copy& cp : in)
        if (cp.bytes && cp.from && cudaMemcpyAsync(const_cast<void*>(cp.to), cp.from, cp.bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
            return SAN_ERR_CUDA;
    const int32_t rc = san_decode_step(ctx, d, stream);
    if (rc != SAN_OK) return rc;
    for (const Copy& cp : out)      // S comes back only if the host asked for it and the device step stored it
        if (cp.bytes && cp.from && cp.to && cudaMemcpyAsync(const_cast<void*>(cp.to), cp.from, cp.bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return SAN_ERR_CUDA;
    return SAN_OK;
}

int32_t san_beam_reorder(san_ctx* ctx, const int32_t* d_sent_ids, const int32_t* d_parent,
                         const int32_t* d_lens, int32_t n_sent, int32_t max_len, void* stream) {
    if (!ctx || !d_sent_ids || !d_parent || !d_lens) return SAN_ERR_NULL;
    const san_config& c = ctx->cfg;
    if (n_sent < 0 || n_sent > c.max_sent) return SAN_ERR_SHAPE;
    if (max_len == 0) max_len = c.max_tgt_len;
    if (max_len < 1 || max_len > c.max_tgt_len) return SAN_ERR_SHAPE;
    if (n_sent == 0) return SAN_OK;
    ReorderParams p;
    std::memset(&p, 0, sizeof(p));
    p.sent_ids = d_sent_ids; p.parent = d_parent; p.lens = d_lens;
    p.n_sent = n_sent; p.beam = c.beam; p.max_sent = c.max_sent; p.max_units = max_len; p.err = ctx->err;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto launch = [&](const ReorderParams& q) -> int32_t {
        const long long gx = (long long)q.tiles_per_panel * q.n_heads * q.n_sent;
        if (gx > 0x7fffffffLL || q.n_planes > 65535) return SAN_ERR_SHAPE;
        if (q.beam <= 8) beam_reorder_kernel<8><<<dim3((unsigned)gx, (unsigned)q.n_planes), kReorderThreads, 0, st>>>(q);
        else beam_reorder_kernel<SAN_MAX_BEAM><<<dim3((unsigned)gx, (unsigned)q.n_planes), kReorderThreads, 0, st>>>(q);
        return cuda_status(cudaGetLastError());
    };
    if (c.self_is_aan) {       // the running sums [layer][sequence][H*64] float32
        p.base = ctx->cache + ctx->off_aan; p.plane_bytes = (long long)ctx->aan_plane_bytes;
        p.n_planes = c.n_layers; p.n_heads = 1; p.head_bytes = 0;
        p.fixed_pieces = c.n_heads * kDh * (int)sizeof(float) / 16;
        p.seq_bytes = (long long)p.fixed_pieces * 16;
        p.tiles_per_panel = ceil_div(p.fixed_pieces, kReorderThreads);
        return launch(p);
    }
    // key planes of the blocks and value planes of the layers, same geometry
    const int row_bytes = kDh * ctx->elem_bytes;
    p.n_heads = c.n_heads; p.plane_bytes = (long long)ctx->self_plane_bytes;
    p.head_bytes = (long long)c.max_tgt_len * row_bytes;
    p.seq_bytes = p.head_bytes * c.n_heads;
    p.unit_pieces = row_bytes / 16;
    if ((long long)max_len * p.unit_pieces > 0x7fffffffLL) return SAN_ERR_SHAPE;
    p.tiles_per_panel = ceil_div(max_len * p.unit_pieces, kReorderThreads);
    p.base = ctx->cache + ctx->off_self_k; p.n_planes = ctx->self_pol.n_blocks + ctx->n_self_v_planes;
    if (ctx->self_pol.n_blocks < ctx->n_self_k_planes) {
        // the policy in force uses fewer key planes than the arena holds: the unused planes lie
        // between the used key planes and the value planes, so the two runs are launched apart
        p.n_planes = ctx->self_pol.n_blocks;
        const int32_t rc = launch(p);
        if (rc != SAN_OK) return rc;
        p.base = ctx->cache + ctx->off_self_v; p.n_planes = ctx->n_self_v_planes;
    }
    return launch(p);
}

int32_t san_full_block(int32_t dtype, int32_t n_heads, int32_t n_layers, int32_t causal, const void* d_q,
                       const void* d_k, const void* d_v, const int32_t* d_lens, int32_t n_seq, int32_t cap_len,
                       int32_t max_len, float* d_S, int64_t ld_s, void* d_out, void* stream) {
    if (!d_q || !d_k || !d_v || !d_lens || !d_out) return SAN_ERR_NULL;
    if (dtype != SAN_BF16) return dtype == SAN_F32 ? SAN_ERR_UNSUPPORTED : SAN_ERR_DTYPE;
    if (n_heads < 1 || n_heads > 65535 || n_layers < 1 || n_layers > SAN_MAX_LAYERS) return SAN_ERR_SHAPE;
    if (n_seq < 0 || n_seq > 65535 || cap_len < 1) return SAN_ERR_SHAPE;
    if (max_len == 0) max_len = cap_len;
    if (max_len < 1 || max_len > cap_len) return SAN_ERR_SHAPE;
    const bool tc5 = max_len >= kTcQ && n_layers <= kTcMaxLayers;      // sequences that fill a 128-query tile
    if (!tc5 && max_len > kFullMaxLen) return SAN_ERR_UNSUPPORTED;      // the mma.sync kernel keeps a row of scores per query on chip
    if (d_S && ld_s < max_len) return SAN_ERR_SHAPE;
    if (n_seq == 0) return SAN_OK;
    FullParams p;
    p.q = static_cast<const __nv_bfloat16*>(d_q); p.k = static_cast<const __nv_bfloat16*>(d_k);
    p.v = static_cast<const __nv_bfloat16*>(d_v); p.out = static_cast<__nv_bfloat16*>(d_out);
    p.S = d_S; p.ld_s = ld_s; p.lens = d_lens;
    p.layer_elems = (long long)n_seq * cap_len * n_heads * kDh;
    p.n_seq = n_seq; p.H = n_heads; p.cap = cap_len; p.max_len = max_len; p.n_layers = n_layers; p.causal = causal ? 1 : 0;
    p.strip_ld = (int)align_up((size_t)max_len, kFullChunk) + 8;
    p.scale_log2e = (float)(1.4426950408889634 / std::sqrt((double)kDh));
    // the opt-in above 48 KB of dynamic shared memory is a per-device attribute of a kernel:
    // remember the largest value set on each device (it only ever needs to grow)
    auto opt_in = [](const void* fn, size_t bytes, size_t* set_per_device) -> bool {
        if (bytes <= 48 * 1024) return true;
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return false;
        if (dev < 0 || dev >= 64 || bytes > set_per_device[dev]) {
            if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) return false;
            if (dev >= 0 && dev < 64) set_per_device[dev] = bytes;
        }
        return true;
    };
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (tc5) {
        // tcgen05 path, accumulators in tensor memory; keys stream in chunks, so any length goes
        static size_t set_tc5[64] = {};
        const size_t smem = full_tc5_smem_bytes();
        if (!opt_in((const void*)full_block_tc5_kernel, smem, set_tc5)) return SAN_ERR_CUDA;
        const dim3 grid((unsigned)ceil_div(max_len, kTcQ), (unsigned)n_heads, (unsigned)n_seq);
        full_block_tc5_kernel<<<grid, kTcThreads, smem, st>>>(p);
        return cuda_status(cudaGetLastError());
    }
    static size_t set_mma[64] = {};
    const size_t smem = (size_t)kFullChunk * kFullRowBytes + (size_t)4 * 16 * p.strip_ld * sizeof(float);
    if (!opt_in((const void*)full_block_kernel, smem, set_mma)) return SAN_ERR_CUDA;
    const dim3 grid((unsigned)ceil_div(max_len, kFullQ), (unsigned)n_heads, (unsigned)n_seq);
    full_block_kernel<<<grid, 128, smem, st>>>(p);
    return cuda_status(cudaGetLastError());
}

int32_t san_js_matrix(int32_t n_layers, const float* d_S, int64_t layer_stride, int64_t ld_s,
                      int32_t n_rows, int32_t n_heads, const int32_t* d_lens, double* d_js, void* stream) {
    if (!d_S || !d_lens || !d_js) return SAN_ERR_NULL;
    if (n_layers < 1 || n_layers > SAN_MAX_LAYERS) return SAN_ERR_SHAPE;
    if (n_rows < 0 || n_heads < 1 || ld_s < 1 || layer_stride < 0) return SAN_ERR_SHAPE;
    if (n_layers > 1 && layer_stride < (int64_t)n_rows * n_heads * ld_s) return SAN_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(d_js, 0, sizeof(double) * n_layers * n_layers, st) != cudaSuccess) return SAN_ERR_CUDA;
    const long long warps = (long long)n_rows * n_heads;
    if (warps > 0 && n_layers > 1) {
        JsParams p;
        p.S = d_S; p.layer_stride = layer_stride; p.ld = ld_s; p.lens = d_lens;
        p.n_layers = n_layers; p.n_rows = n_rows; p.n_heads = n_heads; p.js = d_js;
        const long long grid = (warps + 7) / 8;
        if (grid > 0x7fffffffLL) return SAN_ERR_SHAPE;
        js_pairs_kernel<<<(unsigned)grid, 256, 0, st>>>(p);
        if (cudaGetLastError() != cudaSuccess) return SAN_ERR_CUDA;
    }
    js_finish_kernel<<<n_layers, n_layers, 0, st>>>(d_js, n_layers, (double)warps);
    return cuda_status(cudaGetLastError());
}

int32_t san_block_similarity(const double* js, int32_t n_layers, int32_t m, int32_t n, double* sim) {
    if (!js || !sim) return SAN_ERR_NULL;
    if (n_layers < 1 || n_layers > SAN_MAX_LAYERS) return SAN_ERR_SHAPE;
    if (m < 0 || n >= n_layers || m >= n) return SAN_ERR_RANGE;
    *sim = block_similarity(js, n_layers, m, n);
    return SAN_OK;
}

int32_t san_policy_search(const double* js, int32_t n_layers, double theta, int32_t* sizes, int32_t* n_blocks) {
    if (!js || !sizes || !n_blocks) return SAN_ERR_NULL;
    if (n_layers < 1 || n_layers > SAN_MAX_LAYERS) return SAN_ERR_SHAPE;
    if (!(theta == theta)) return SAN_ERR_RANGE;      // NaN compares false with everything
    *n_blocks = search_policy(js, n_layers, theta, sizes);
    return SAN_OK;
}

int32_t san_device_status(san_ctx* ctx, int32_t* first_error, int32_t* detail, void* stream) {
    if (!ctx || !first_error) return SAN_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int words[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    cudaError_t e = cudaMemcpyAsync(words, ctx->err, sizeof(words), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e == cudaSuccess && words[0] != 0) {
        // A step that stopped early (a wait ran out) may have left tickets of split rows part-way:
        // clear them with the error words, or later rows would never see their last span arrive.
        const size_t clear = words[0] == SAN_ERR_TIMEOUT ? ctx->ws_off_part : sizeof(words);
        e = cudaMemsetAsync(ctx->err, 0, clear, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    }
    if (e != cudaSuccess) return SAN_ERR_CUDA;
    *first_error = words[0];
    if (detail) for (int i = 0; i < 4; ++i) detail[i] = words[1 + i];
    return SAN_OK;
}

const char* san_status_string(int32_t status) {
    switch (status) {
        case SAN_OK: return "ok";
        case SAN_ERR_NULL: return "a required pointer is NULL";
        case SAN_ERR_SHAPE: return "a size or count is out of range";
        case SAN_ERR_POLICY: return "invalid sharing policy";
        case SAN_ERR_CAPACITY: return "a buffer is too small or the policy has more blocks than key planes";
        case SAN_ERR_DTYPE: return "unknown element type";
        case SAN_ERR_RANGE: return "layer, block or position outside the allowed range";
        case SAN_ERR_CUDA: return "a CUDA runtime call failed";
        case SAN_ERR_DEVICE_CHECK: return "a kernel skipped an item with an invalid id, length or position";
        case SAN_ERR_TIMEOUT: return "a bounded device wait ran out";
        case SAN_ERR_UNSUPPORTED: return "not supported by this configuration";
        default: return "unknown status";
    }
}

}  // extern "C"
