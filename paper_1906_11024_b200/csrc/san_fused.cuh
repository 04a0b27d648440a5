// One decode step in one launch: cache append, weights (Eq. 1) and apply (Eq. 2 with Eq. 4)
// for every block of both attention kinds, plus the AAN running average.
//
// Every (kind, block, item, head[, span]) is independent, so the step is a flat list of
// work items drained by persistent warps.  Each warp owns a ring of shared-memory stages
// fed by bulk asynchronous copies (cp.async.bulk, completion on an mbarrier): the query
// rows, then the key panel in tiles, then the value panel of every layer of the block in
// tiles.  Copies are issued up to kFusedStages tiles ahead of their use and run on into
// the next item, so the loads of an item never wait for the arithmetic of the one before.
// For self-attention the newest position is not in the cache yet: its key/value rows are
// copied from the caller's k_new/v_new into the last tile beside the cached rows, and
// written to the cache from there.  S never leaves the chip between weights and apply
// (it is also written out for the caller).
#pragma once

#include "san_kernels.cuh"

namespace san {

constexpr int kStageBytes = 4096;   // one tile: 32 bf16 rows or 16 float32 rows
constexpr int kFusedWarps = 12;
constexpr int kFusedStages = 4;
constexpr int kZFloats = 512;       // scores a warp keeps on chip: span <= kZFloats / NQ
constexpr int kDescSlots = 4;       // decoded items a warp may have in flight
constexpr int kMaxSpans = 32;

enum { TAG_STEP = 6 };

struct StepParams {
    // decoder self-attention (absent when n_self_blocks == 0)
    const char* q_self; const char* k_new; const char* v_new;   // [N_s][n][H][64], same, [M][n][H][64]
    const int* seq_ids; const int* pos;                         // row written this step; length = pos + 1
    float* S_self; long long ld_t; char* O_self;                // S may be null
    int n_seqs, max_len;
    // encoder-decoder attention
    const char* q_enc;                                          // [N_e][n_sent][beam][H][64]
    const int* sent_ids; const int* src_lens;
    float* S_enc; long long ld_s; char* O_enc;
    int n_sent, max_src;
    // AAN in place of self-attention (absent when x_aan == null)
    const char* x_aan; const int* t_aan; float* aan_sum; int n_aan_layers;
    // geometry
    int H, beam, n_self_blocks, n_enc_blocks, cap_tgt, cap_src, max_seqs, max_sent, enc_v_by_block;
    char* selfK; char* selfV; char* memK; char* memV;
    long long self_plane_bytes, mem_plane_bytes;
    int self_span, self_nspans, enc_span, enc_nspans;           // positions per item, spans per row at the bound
    long long n_enc_items, n_items;                             // enc items come first in the list
    long long self_part_base;                                   // float offset of the self rows' partials
    int enc_part_stride, self_part_stride;                      // floats per (row, span)
    float* part; int* tickets; int* err;
    float scale_log2e;
    unsigned char self_first[SAN_MAX_LAYERS], self_size[SAN_MAX_LAYERS];
    unsigned char enc_first[SAN_MAX_LAYERS], enc_size[SAN_MAX_LAYERS];
};

// A decoded work item, kept in shared memory between the copy side and the math side.
struct ItemDesc {
    const char* q; long long q_stride;        // query row qi at q + qi*q_stride
    const char* Kp;                           // key panel, row 0
    const char* Vp; long long v_plane;        // value panel of the block's first layer, row 0
    const char* knew; const char* vnew; long long vnew_stride;   // newest rows (self only)
    float* S; long long S_qstride;            // S row of query 0 (may be null)
    char* O; long long O_lstride, O_qstride;  // output of (first layer, query 0)
    long long row_id;                         // ticket index of the row
    float* part;                              // partial sums of this (row, span)
    int kind, nq, pi, len, j0, j1, n_spans, span, n_pos_tiles, n_tiles, has_new, part_stride;
};

// ------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after about a second and reports it; never spins for ever.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > 2000000000LL) return false;
    }
    return true;
}

template <typename T> struct FusedGeom {
    static constexpr int ROW_BYTES = kDh * (int)sizeof(T);
    static constexpr int TR = kStageBytes / ROW_BYTES;   // rows per tile
};

// ------------------------------------------------------------------------------ the kernel
template <typename T>
struct FusedWarp {
    using G = RowGeom<T>;
    using F = FusedGeom<T>;
    static constexpr int VEC = G::VEC, LPR = G::LPR, RPW = 32 / LPR, ROW_BYTES = F::ROW_BYTES, TR = F::TR;

    const StepParams& p;
    char* ring;            // kFusedStages stages of this warp
    uint64_t* bars;        // one per stage
    float* zs;             // kZFloats scores
    ItemDesc* descs;       // kDescSlots
    int lane, g, c;
    long long stride;      // warps in the grid
    // copy side
    long long p_item; int p_tile; unsigned p_seq; unsigned p_n;   // next item / tile to issue; tiles issued; items decoded
    int pre_id, pre_len;   // metadata of p_item, fetched ahead
    // math side
    unsigned c_seq, c_n;
    bool dead;             // a wait ran out: stop issuing, drain, leave

    __device__ FusedWarp(const StepParams& pp) : p(pp) {}

    // ---- item list: [enc items][self items]; within a kind: ((block, item, head), span)
    __device__ void fetch_meta(long long it, int* id, int* len) const {
        if (it >= p.n_items) { *id = 0; *len = 0; return; }
        if (it < p.n_enc_items) {
            const long long row = it / p.enc_nspans;
            const int item = (int)((row / p.H) % p.n_sent);
            *id = p.sent_ids[item]; *len = p.src_lens[item];
        } else {
            const long long row = (it - p.n_enc_items) / p.self_nspans;
            const int item = (int)((row / p.H) % p.n_seqs);
            *id = p.seq_ids[item]; *len = p.pos[item] + 1;
        }
    }

    // Decodes item `it` into *d; returns false if the item is to be skipped.
    __device__ bool decode(long long it, int id, int len, ItemDesc* d) const {
        const bool enc = it < p.n_enc_items;
        const long long local = enc ? it : it - p.n_enc_items;
        const int nspans_max = enc ? p.enc_nspans : p.self_nspans;
        const int span_len = enc ? p.enc_span : p.self_span;
        const int span = (int)(local % nspans_max);
        const long long row = local / nspans_max;
        const int h = (int)(row % p.H);
        const int n_it = enc ? p.n_sent : p.n_seqs;
        const int item = (int)((row / p.H) % n_it);
        const int block = (int)(row / ((long long)p.H * n_it));
        const int max_ids = enc ? p.max_sent : p.max_seqs;
        const int bound = enc ? p.max_src : p.max_len;
        const bool reporter = (lane == 0 && span == 0 && h == 0 && block == 0);
        if (id < 0 || id >= max_ids) { if (reporter) record_error(p.err, TAG_STEP, item, id, max_ids); return false; }
        if (len < 1 || len > bound) { if (reporter) record_error(p.err, TAG_STEP, item, len, bound); return false; }
        const int j0 = span * span_len;
        if (j0 >= len) return false;                      // a shorter row has fewer spans
        if (lane != 0) return true;                       // one lane fills the descriptor
        const int j1 = min(len, j0 + span_len);
        const int nq = enc ? p.beam : 1;
        const int first = enc ? p.enc_first[block] : p.self_first[block];
        const int pi = enc ? (p.enc_v_by_block ? 1 : p.enc_size[block]) : p.self_size[block];
        const int cap = enc ? p.cap_src : p.cap_tgt;
        const long long plane = enc ? p.mem_plane_bytes : p.self_plane_bytes;
        const long long panel = (((long long)id * p.H + h) * cap) * ROW_BYTES;
        d->kind = enc ? 1 : 0; d->nq = nq; d->pi = pi; d->len = len; d->j0 = j0; d->j1 = j1;
        d->n_spans = (len + span_len - 1) / span_len; d->span = span;
        d->n_pos_tiles = (j1 - j0 + TR - 1) / TR;
        d->n_tiles = 1 + d->n_pos_tiles * (1 + pi);
        d->has_new = (!enc && j1 == len) ? 1 : 0;
        d->row_id = enc ? row : (p.n_enc_items / p.enc_nspans) + row;
        d->part_stride = enc ? p.enc_part_stride : p.self_part_stride;
        d->part = p.part + (enc ? 0 : p.self_part_base) + (row * nspans_max + span) * (long long)d->part_stride;
        if (enc) {
            d->q = p.q_enc + ((((long long)block * p.n_sent + item) * nq) * p.H + h) * ROW_BYTES;
            d->q_stride = (long long)p.H * ROW_BYTES;
            d->Kp = p.memK + block * plane + panel;
            d->Vp = p.memV + (p.enc_v_by_block ? block : first) * plane + panel;
            d->knew = nullptr; d->vnew = nullptr; d->vnew_stride = 0;
            d->S = p.S_enc ? p.S_enc + ((((long long)block * p.n_sent + item) * nq) * p.H + h) * p.ld_s : nullptr;
            d->S_qstride = (long long)p.H * p.ld_s;
            const int o_first = p.enc_v_by_block ? block : first;
            d->O = p.O_enc + ((((long long)o_first * p.n_sent + item) * nq) * p.H + h) * ROW_BYTES;
            d->O_lstride = (long long)p.n_sent * nq * p.H * ROW_BYTES;
            d->O_qstride = (long long)p.H * ROW_BYTES;
        } else {
            const long long in_row = ((long long)item * p.H + h) * ROW_BYTES;
            const long long in_layer = (long long)p.n_seqs * p.H * ROW_BYTES;
            d->q = p.q_self + block * in_layer + in_row; d->q_stride = 0;
            d->Kp = p.selfK + block * plane + panel;
            d->Vp = p.selfV + first * plane + panel;
            d->knew = p.k_new + block * in_layer + in_row;
            d->vnew = p.v_new + first * in_layer + in_row; d->vnew_stride = in_layer;
            d->S = p.S_self ? p.S_self + (((long long)block * p.n_seqs + item) * p.H + h) * p.ld_t : nullptr;
            d->S_qstride = 0;
            d->O = p.O_self + first * in_layer + in_row;
            d->O_lstride = in_layer; d->O_qstride = 0;
        }
        d->v_plane = plane;
        return true;
    }

    // Moves the copy side to the next item that is not skipped and decodes it.
    __device__ void next_item() {
        while (p_item < p.n_items) {
            ItemDesc* d = &descs[p_n % kDescSlots];
            const bool ok = decode(p_item, pre_id, pre_len, d);
            if (ok) {
                __syncwarp();
                p_n += 1; p_tile = 0;
                fetch_meta(p_item + stride, &pre_id, &pre_len);   // used when this item's tiles are all issued
                return;
            }
            p_item += stride;
            fetch_meta(p_item, &pre_id, &pre_len);
        }
    }

    // Issues the copies of one tile of the item being produced, if any is left.
    __device__ void produce() {
        if (dead || p_item >= p.n_items) return;
        if (lane == 0) {
            const ItemDesc& d = descs[(p_n - 1) % kDescSlots];
            const unsigned s = p_seq % kFusedStages;
            char* dst = ring + s * kStageBytes;
            uint64_t* bar = bars + s;
            if (p_tile == 0) {
                mbar_expect_tx(bar, (uint32_t)(d.nq * ROW_BYTES));
                for (int qi = 0; qi < d.nq; ++qi) bulk_g2s(dst + qi * ROW_BYTES, d.q + qi * d.q_stride, ROW_BYTES, bar);
            } else {
                const int u = p_tile - 1;
                const int which = u / d.n_pos_tiles, ct = u % d.n_pos_tiles;
                const int s0 = d.j0 + ct * TR;
                const int r = min(TR, d.j1 - s0);
                const bool with_new = d.has_new && (s0 + r == d.len);
                const int r_cache = with_new ? r - 1 : r;
                const char* src = (which == 0 ? d.Kp : d.Vp + (long long)(which - 1) * d.v_plane) + (long long)s0 * ROW_BYTES;
                mbar_expect_tx(bar, (uint32_t)(r * ROW_BYTES));
                if (r_cache > 0) bulk_g2s(dst, src, (uint32_t)(r_cache * ROW_BYTES), bar);
                if (with_new) {
                    const char* nsrc = which == 0 ? d.knew : d.vnew + (long long)(which - 1) * d.vnew_stride;
                    bulk_g2s(dst + r_cache * ROW_BYTES, nsrc, ROW_BYTES, bar);
                }
            }
        }
        p_seq += 1; p_tile += 1;
        const int n_tiles = descs[(p_n - 1) % kDescSlots].n_tiles;
        if (p_tile == n_tiles) { p_item += stride; next_item(); }
    }

    // Waits for the next tile in order; returns its stage or null after a timeout.
    __device__ const char* acquire() {
        const unsigned s = c_seq % kFusedStages;
        if (!mbar_wait(bars + s, (c_seq / kFusedStages) & 1)) {
            if (lane == 0) { if (atomicCAS(&p.err[0], 0, (int)SAN_ERR_TIMEOUT) == 0) { p.err[1] = TAG_STEP; p.err[2] = (int)c_seq; } }
            dead = true;
            return nullptr;
        }
        return ring + s * kStageBytes;
    }
    // Every lane is done with the tile: hand the stage back to the copy side.
    __device__ void release() {
        __syncwarp();
        c_seq += 1;
        produce();
    }

    template <int NQ> __device__ bool process(const ItemDesc& d);
    __device__ void drain();
};

// After a timeout: the copies already issued may still land in this warp's stages, so give
// each a last bounded chance to finish before the CTA's shared memory can go away.
template <typename T>
__device__ void FusedWarp<T>::drain() {
    while (c_seq != p_seq) {
        const unsigned s = c_seq % kFusedStages;
        const uint32_t par = (c_seq / kFusedStages) & 1;
        const long long t0 = clock64();
        while (!mbar_try_wait(bars + s, par)) { if (clock64() - t0 > 200000000LL) break; }
        c_seq += 1;
    }
}

template <typename T>
template <int NQ>
__device__ bool FusedWarp<T>::process(const ItemDesc& d) {
    constexpr int UNROLL = 4;
    constexpr int ZQ = kZFloats / NQ;          // score slots per query row
    const int n = d.j1 - d.j0;
    const int nq = d.nq;

    // ---- tile 0: the query rows
    float qf[NQ][VEC];
    {
        const char* st = acquire();
        if (!st) return false;
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) {
            if (qi < nq) {
                unpack16<T>(*reinterpret_cast<const uint4*>(st + qi * ROW_BYTES + c * 16), qf[qi]);
#pragma unroll
                for (int e = 0; e < VEC; ++e) qf[qi][e] *= p.scale_log2e;
            } else {
#pragma unroll
                for (int e = 0; e < VEC; ++e) qf[qi][e] = 0.f;
            }
        }
        release();
    }

    // ---- key tiles: scores into zs
    for (int ct = 0; ct < d.n_pos_tiles; ++ct) {
        const char* st = acquire();
        if (!st) return false;
        const int r = min(TR, n - ct * TR);
        const bool with_new = d.has_new && (ct == d.n_pos_tiles - 1);
#pragma unroll
        for (int jb = 0; jb < TR; jb += RPW * UNROLL) {
            if (jb < r) {
                uint4 kv[UNROLL];
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int j = jb + u * RPW + g;
                    kv[u] = (j < r) ? *reinterpret_cast<const uint4*>(st + j * ROW_BYTES + c * 16) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int j = jb + u * RPW + g;
                    float kf[VEC];
                    unpack16<T>(kv[u], kf);
#pragma unroll
                    for (int qi = 0; qi < NQ; ++qi) {
                        float dot = 0.f;
#pragma unroll
                        for (int e = 0; e < VEC; ++e) dot = fmaf(qf[qi][e], kf[e], dot);
#pragma unroll
                        for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                        if (c == 0 && j < r) zs[qi * ZQ + ct * TR + j] = dot;
                    }
                    // the newest key row goes into the cache from here
                    if (with_new && j == r - 1)
                        *reinterpret_cast<uint4*>(const_cast<char*>(d.Kp) + (long long)(d.len - 1) * ROW_BYTES + c * 16) = kv[u];
                }
            }
        }
        release();
    }

    // ---- softmax over the span (log2 domain)
    float part_m[NQ], part_l[NQ];
#pragma unroll
    for (int qi = 0; qi < NQ; ++qi) {
        part_m[qi] = 0.f; part_l[qi] = 1.f;
        if (qi < nq) {
            float m = -INFINITY;
            for (int jj = lane; jj < n; jj += 32) m = fmaxf(m, zs[qi * ZQ + jj]);
            m = warp_max(m);
            float s = 0.f;
            for (int jj = lane; jj < n; jj += 32) { const float e = exp2f(zs[qi * ZQ + jj] - m); zs[qi * ZQ + jj] = e; s += e; }
            s = warp_sum(s);
            part_m[qi] = m; part_l[qi] = s;
            float* Srow = d.S ? d.S + qi * d.S_qstride + d.j0 : nullptr;
            if (d.n_spans == 1) {
                for (int jj = lane; jj < n; jj += 32) {
                    const float w = zs[qi * ZQ + jj] / s;
                    zs[qi * ZQ + jj] = w;
                    if (Srow) Srow[jj] = w;
                }
            } else if (Srow) {
                for (int jj = lane; jj < n; jj += 32) Srow[jj] = zs[qi * ZQ + jj];
            }
        }
    }
    __syncwarp();

    // ---- value tiles, layer by layer
    float* part = d.part;
    for (int l = 0; l < d.pi; ++l) {
        float acc[NQ][VEC];
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi)
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[qi][e] = 0.f;
        for (int ct = 0; ct < d.n_pos_tiles; ++ct) {
            const char* st = acquire();
            if (!st) return false;
            const int r = min(TR, n - ct * TR);
            const bool with_new = d.has_new && (ct == d.n_pos_tiles - 1);
#pragma unroll
            for (int jb = 0; jb < TR; jb += RPW * UNROLL) {
                if (jb < r) {
                    uint4 vv[UNROLL];
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) {
                        const int j = jb + u * RPW + g;
                        vv[u] = (j < r) ? *reinterpret_cast<const uint4*>(st + j * ROW_BYTES + c * 16) : make_uint4(0, 0, 0, 0);
                    }
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) {
                        const int j = jb + u * RPW + g;
                        if (j < r) {
                            float vf[VEC];
                            unpack16<T>(vv[u], vf);
#pragma unroll
                            for (int qi = 0; qi < NQ; ++qi) {
                                const float s = (qi < nq) ? zs[qi * ZQ + ct * TR + j] : 0.f;
#pragma unroll
                                for (int e = 0; e < VEC; ++e) acc[qi][e] = fmaf(s, vf[e], acc[qi][e]);
                            }
                            if (with_new && j == r - 1)
                                *reinterpret_cast<uint4*>(const_cast<char*>(d.Vp) + (long long)l * d.v_plane +
                                                          (long long)(d.len - 1) * ROW_BYTES + c * 16) = vv[u];
                        }
                    }
                }
            }
            release();
        }
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi)
#pragma unroll
            for (int e = 0; e < VEC; ++e)
#pragma unroll
                for (int o = LPR; o < 32; o <<= 1) acc[qi][e] += __shfl_xor_sync(0xffffffffu, acc[qi][e], o);
        if (g == 0) {
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) {
                if (qi < nq) {
                    if (d.n_spans == 1) {
                        *reinterpret_cast<uint4*>(d.O + l * d.O_lstride + qi * d.O_qstride + c * 16) = pack16<T>(acc[qi]);
                    } else {
                        float* pp = part + 2 * NQ + ((long long)l * NQ + qi) * kDh + c * VEC;
#pragma unroll
                        for (int e = 0; e < VEC; ++e) pp[e] = acc[qi][e];
                    }
                }
            }
        }
    }
    if (d.n_spans == 1) return true;

    // ---- split row: park (max, sum); the last span to arrive combines all of them
    if (lane == 0) {
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) { part[qi] = part_m[qi]; part[NQ + qi] = part_l[qi]; }
    }
    __threadfence();
    __syncwarp();
    int t = 0;
    if (lane == 0) t = atomicAdd(p.tickets + d.row_id, 1);
    t = __shfl_sync(0xffffffffu, t, 0);
    if (t != d.n_spans - 1) return true;
    __threadfence();
    const float* row_part = part - (long long)d.span * d.part_stride;
    const int span_len = d.kind ? p.enc_span : p.self_span;
    for (int qi = 0; qi < nq; ++qi) {
        // lane sp holds span sp's weight exp2(m_sp - M) / total
        float m = -INFINITY, l = 0.f;
        if (lane < d.n_spans) { m = __ldcg(row_part + (long long)lane * d.part_stride + qi); l = __ldcg(row_part + (long long)lane * d.part_stride + NQ + qi); }
        const float M = warp_max(m);
        const float wl = (lane < d.n_spans) ? l * exp2f(m - M) : 0.f;
        const float tot = warp_sum(wl);
        const float wgt = (lane < d.n_spans) ? exp2f(m - M) / tot : 0.f;
        if (d.S) {
            float* Srow = d.S + qi * d.S_qstride;
            for (int sp = 0; sp < d.n_spans; ++sp) {
                const float f = __shfl_sync(0xffffffffu, wgt, sp);
                const int b = sp * span_len, e = min(d.len, b + span_len);
                for (int j = b + lane; j < e; j += 32) Srow[j] = __ldcg(Srow + j) * f;
            }
        }
        for (int ly = 0; ly < d.pi; ++ly) {
            float a0 = 0.f, a1 = 0.f;
            for (int sp = 0; sp < d.n_spans; ++sp) {
                const float f = __shfl_sync(0xffffffffu, wgt, sp);
                const float* pp = row_part + (long long)sp * d.part_stride + 2 * NQ + ((long long)ly * NQ + qi) * kDh;
                a0 = fmaf(f, __ldcg(pp + lane), a0);
                a1 = fmaf(f, __ldcg(pp + 32 + lane), a1);
            }
            T* op = reinterpret_cast<T*>(d.O + ly * d.O_lstride + qi * d.O_qstride);
            op[lane] = (T)a0;
            op[32 + lane] = (T)a1;
        }
    }
    if (lane == 0) p.tickets[d.row_id] = 0;
    return true;
}

constexpr size_t fused_smem_bytes() {
    return (size_t)kFusedWarps * (kFusedStages * kStageBytes + kZFloats * sizeof(float) + kDescSlots * sizeof(ItemDesc) +
                                  kFusedStages * sizeof(uint64_t)) + 128;
}

template <typename T, int NQE>
__global__ void __launch_bounds__(kFusedWarps * 32, 1) decode_step_kernel(const __grid_constant__ StepParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    // ---- AAN running average (Table 6 pairing): element-wise, every thread of the grid
    if (p.x_aan) {
        const int d = p.H * kDh, d4 = d >> 2;
        const long long total = (long long)p.n_aan_layers * p.n_seqs * d4;
        for (long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x; u < total; u += (long long)gridDim.x * blockDim.x) {
            const int c4 = (int)(u % d4);
            const int item = (int)((u / d4) % p.n_seqs);
            const int lr = (int)(u / ((long long)d4 * p.n_seqs));
            const int id = p.seq_ids[item], t = p.t_aan[item];
            if (id < 0 || id >= p.max_seqs) { if (c4 == 0 && lr == 0) record_error(p.err, TAG_AAN, item, id, p.max_seqs); continue; }
            if (t < 1 || t > p.cap_tgt) { if (c4 == 0 && lr == 0) record_error(p.err, TAG_AAN, item, t, p.cap_tgt); continue; }
            const long long io = ((long long)lr * p.n_seqs + item) * d + c4 * 4;
            float xv[4];
            if (sizeof(T) == 2) {
                const uint2 raw = *reinterpret_cast<const uint2*>(p.x_aan + io * 2);
                xv[0] = __uint_as_float(raw.x << 16); xv[1] = __uint_as_float(raw.x & 0xffff0000u);
                xv[2] = __uint_as_float(raw.y << 16); xv[3] = __uint_as_float(raw.y & 0xffff0000u);
            } else {
                const float4 raw = *reinterpret_cast<const float4*>(p.x_aan + io * 4);
                xv[0] = raw.x; xv[1] = raw.y; xv[2] = raw.z; xv[3] = raw.w;
            }
            float4* sp = reinterpret_cast<float4*>(p.aan_sum + ((long long)lr * p.max_seqs + id) * d + c4 * 4);
            float4 s = (t == 1) ? make_float4(0.f, 0.f, 0.f, 0.f) : *sp;
            s.x += xv[0]; s.y += xv[1]; s.z += xv[2]; s.w += xv[3];
            *sp = s;
            const float ft = (float)t;
            const float o[4] = {s.x / ft, s.y / ft, s.z / ft, s.w / ft};
            if (sizeof(T) == 2) {
                __nv_bfloat162 a = __floats2bfloat162_rn(o[0], o[1]), b = __floats2bfloat162_rn(o[2], o[3]);
                uint2 r; r.x = *reinterpret_cast<uint32_t*>(&a); r.y = *reinterpret_cast<uint32_t*>(&b);
                *reinterpret_cast<uint2*>(p.O_self + io * 2) = r;
            } else {
                *reinterpret_cast<float4*>(p.O_self + io * 4) = make_float4(o[0], o[1], o[2], o[3]);
            }
        }
    }
    if (p.n_items == 0) return;

    // ---- attention items
    FusedWarp<T> w(p);
    char* base = reinterpret_cast<char*>(smem);
    w.ring = base + (size_t)warp * kFusedStages * kStageBytes;
    char* after = base + (size_t)kFusedWarps * kFusedStages * kStageBytes;
    w.zs = reinterpret_cast<float*>(after) + (size_t)warp * kZFloats;
    after += (size_t)kFusedWarps * kZFloats * sizeof(float);
    w.descs = reinterpret_cast<ItemDesc*>(after) + (size_t)warp * kDescSlots;
    after += (size_t)kFusedWarps * kDescSlots * sizeof(ItemDesc);
    w.bars = reinterpret_cast<uint64_t*>(after) + (size_t)warp * kFusedStages;
    w.lane = lane; w.g = lane / RowGeom<T>::LPR; w.c = lane % RowGeom<T>::LPR;
    w.stride = (long long)gridDim.x * kFusedWarps;
    w.p_item = (long long)blockIdx.x * kFusedWarps + warp;   // neighbouring items go to different SMs' warps
    w.p_tile = 0; w.p_seq = 0; w.p_n = 0; w.c_seq = 0; w.c_n = 0; w.dead = false;
    if (lane == 0) {
        for (int s = 0; s < kFusedStages; ++s) mbar_init(w.bars + s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    w.fetch_meta(w.p_item, &w.pre_id, &w.pre_len);
    w.next_item();
    for (int s = 0; s < kFusedStages; ++s) w.produce();
    while (w.c_n < w.p_n && !w.dead) {
        const ItemDesc& d = w.descs[w.c_n % kDescSlots];
        const bool ok = d.kind ? w.template process<NQE>(d) : w.template process<1>(d);
        (void)ok;
        w.c_n += 1;
    }
    if (w.dead) w.drain();
}

}  // namespace san
