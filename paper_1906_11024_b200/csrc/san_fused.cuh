// One decode step in one launch: cache append, weights (Eq. 1) and apply (Eq. 2 with Eq. 4)
// for every block of both attention kinds, plus the AAN running average.
//
// Every (kind, block, item, head[, span]) is independent, so the step is a flat list of
// work items (encoder-memory items, the big ones, first).  CTA b owns items b, b+G, b+2G,
// ... (G = CTAs in the grid), so every CTA gets the same mix; its warps take the next one
// from a counter in shared memory.  Each warp owns a ring of shared-memory stages fed by
// bulk asynchronous copies (cp.async.bulk, completion on an mbarrier): the query rows,
// then the key panel in tiles, then the value panel of every layer of the block in tiles.
// Copies are issued several tiles ahead of their use and run on into the next item, so
// the loads of an item never wait for the arithmetic of the one before.  For
// self-attention the newest position is not in the cache yet: its key/value rows are
// copied from the caller's k_new/v_new into the last tile beside the cached rows, and
// written to the cache from there.  S never leaves the chip between weights and apply
// (it is also written out for the caller).  bf16 items run on the tensor cores (mma.sync,
// float32 accumulate) because the step is bound by instruction issue; float32 items use
// packed two-wide FMAs on the CUDA cores.
#pragma once

#include "san_kernels.cuh"

namespace san {

constexpr int kStageBytes = 4096;   // one tile: 32 bf16 rows or 16 float32 rows
constexpr int kFusedWarps = 16;
constexpr int kFusedStages = 3;
constexpr int kZFloats = 256;       // scores a warp keeps on chip: span <= kZFloats / NQ
constexpr int kDescSlots = 6;       // decoded items a warp keeps (in flight, being finished, being decoded)
constexpr int kMaxSpans = 32;

enum { TAG_STEP = 6 };

// Exact division of n < 2^31 by a fixed divisor with one multiply-high (Granlund and
// Montgomery's round-up method): q = (mulhi(n, mul) + n) >> shift.
struct FastDiv {
    unsigned mul, shift, div;
    __device__ __forceinline__ void divmod(unsigned n, unsigned* q, unsigned* r) const {
        *q = (unsigned)(((unsigned long long)__umulhi(n, mul) + n) >> shift);
        *r = n - *q * div;
    }
};

struct StepParams {
    // decoder self-attention
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
    int H, beam, cap_tgt, cap_src, max_seqs, max_sent, enc_v_by_block;
    char* selfK; char* selfV; char* memK; char* memV;
    long long self_plane_bytes, mem_plane_bytes;
    int self_span, self_nspans, enc_span, enc_nspans;           // positions per item, spans per row at the bound
    unsigned n_enc_items, n_items;                              // enc items come first in the list
    unsigned n_enc_rows;
    long long self_part_base;                                   // float offset of the self rows' partials
    int enc_part_stride, self_part_stride;                      // floats per (row, span)
    FastDiv enc_div_span, enc_div_h, enc_div_item, self_div_span, self_div_h, self_div_item;
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
    float* part;                              // partial sums of this (row, span)
    unsigned row_id;                          // ticket index of the row
    int kind, nq, pi, len, j0, j1, n_spans, span, has_new, part_stride;
};

// ------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after about a second and reports it; never spins for ever.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > 2000000000LL) return false;
    }
    return true;
}

// Four 8x8 b16 matrices from shared memory, one row address per lane (plain / transposed).
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <typename T> struct FusedGeom {
    static constexpr int ROW_BYTES = kDh * (int)sizeof(T);
    static constexpr int TR = kStageBytes / ROW_BYTES;   // rows per tile
};

// 16 bytes of a row as packed float pairs
template <typename T> struct Pairs;
template <> struct Pairs<__nv_bfloat16> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void load(const uint4& v, float2* f) {
        f[0] = make_float2(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u));
        f[1] = make_float2(__uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
        f[2] = make_float2(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xffff0000u));
        f[3] = make_float2(__uint_as_float(v.w << 16), __uint_as_float(v.w & 0xffff0000u));
    }
    static __device__ __forceinline__ uint4 store(const float2* f) {
        uint4 v;
        __nv_bfloat162 a = __floats2bfloat162_rn(f[0].x, f[0].y), b = __floats2bfloat162_rn(f[1].x, f[1].y);
        __nv_bfloat162 c = __floats2bfloat162_rn(f[2].x, f[2].y), d = __floats2bfloat162_rn(f[3].x, f[3].y);
        v.x = *reinterpret_cast<uint32_t*>(&a); v.y = *reinterpret_cast<uint32_t*>(&b);
        v.z = *reinterpret_cast<uint32_t*>(&c); v.w = *reinterpret_cast<uint32_t*>(&d);
        return v;
    }
};
template <> struct Pairs<float> {
    static constexpr int N = 2;
    static __device__ __forceinline__ void load(const uint4& v, float2* f) {
        f[0] = make_float2(__uint_as_float(v.x), __uint_as_float(v.y));
        f[1] = make_float2(__uint_as_float(v.z), __uint_as_float(v.w));
    }
    static __device__ __forceinline__ uint4 store(const float2* f) {
        return make_uint4(__float_as_uint(f[0].x), __float_as_uint(f[0].y), __float_as_uint(f[1].x), __float_as_uint(f[1].y));
    }
};

// ------------------------------------------------------------------------------ the warp
template <typename T>
struct FusedWarp {
    using G = RowGeom<T>;
    using F = FusedGeom<T>;
    using P = Pairs<T>;
    static constexpr int VEC = G::VEC, LPR = G::LPR, RPW = 32 / LPR, ROW_BYTES = F::ROW_BYTES, TR = F::TR;
    static constexpr int NP = P::N;          // float pairs per 16 bytes
    static constexpr int BLK = 8;            // rows per inner block
    static constexpr int UN = BLK / RPW;     // loads per lane per block

    const StepParams& p;
    uint32_t ring, bars;   // shared-space addresses: stages and their barriers
    const char* ring_g;    // the same stages through a generic pointer
    float* zs;             // kZFloats floats
    ItemDesc* descs;       // kDescSlots
    unsigned* cta_next;    // shared counter: next slot of this CTA's item sequence to hand out
    int lane, g, c;
    // copy side: the item being issued, the next one (metadata on its way), the one after
    bool p_active;
    unsigned p_seq, p_n;
    int p_which, p_s0, p_j0, p_j1, p_pi, p_q_done;
    const char* p_panel;
    unsigned nx_item; int nx_id, nx_len;      // next item and its prefetched id / length
    unsigned nn_item;                         // the item after that
    // math side
    unsigned c_seq, c_n;
    bool dead;             // a wait ran out: stop issuing, drain, leave

    __device__ FusedWarp(const StepParams& pp) : p(pp) {}

    __device__ __forceinline__ unsigned item_of_slot(unsigned k) const {
        const unsigned long long it = (unsigned long long)k * gridDim.x + blockIdx.x;
        return it < p.n_items ? (unsigned)it : p.n_items;
    }
    __device__ __forceinline__ unsigned grab() {
        unsigned k = 0;
        if (lane == 0) k = atomicAdd(cta_next, 1u);
        return item_of_slot(__shfl_sync(0xffffffffu, k, 0));
    }

    // ---- item list: [enc items][self items]; within a kind: (((block, item), head), span)
    __device__ __forceinline__ void split(unsigned it, bool* enc, unsigned* block, unsigned* item, unsigned* h, unsigned* span,
                                          unsigned* row) const {
        *enc = it < p.n_enc_items;
        unsigned bi;
        if (*enc) {
            p.enc_div_span.divmod(it, row, span);
            p.enc_div_h.divmod(*row, &bi, h);
            p.enc_div_item.divmod(bi, block, item);
        } else {
            p.self_div_span.divmod(it - p.n_enc_items, row, span);
            p.self_div_h.divmod(*row, &bi, h);
            p.self_div_item.divmod(bi, block, item);
        }
    }
    __device__ __forceinline__ void fetch_meta(unsigned it, int* id, int* len) const {
        *id = 0; *len = 0;
        if (it >= p.n_items) return;
        bool enc; unsigned block, item, h, span, row;
        split(it, &enc, &block, &item, &h, &span, &row);
        if (enc) { *id = p.sent_ids[item]; *len = p.src_lens[item]; }
        else { *id = p.seq_ids[item]; *len = p.pos[item] + 1; }
    }

    // Decodes item `it` into *d (lane 0 writes it); returns false if the item is to be skipped.
    __device__ bool decode(unsigned it, int id, int len, ItemDesc* d) const {
        bool enc; unsigned block, item, h, span, row;
        split(it, &enc, &block, &item, &h, &span, &row);
        const int span_len = enc ? p.enc_span : p.self_span;
        const int max_ids = enc ? p.max_sent : p.max_seqs;
        const int bound = enc ? p.max_src : p.max_len;
        const bool reporter = (lane == 0 && span == 0 && h == 0 && block == 0);
        if (id < 0 || id >= max_ids) { if (reporter) record_error(p.err, TAG_STEP, (int)item, id, max_ids); return false; }
        if (len < 1 || len > bound) { if (reporter) record_error(p.err, TAG_STEP, (int)item, len, bound); return false; }
        const int j0 = (int)span * span_len;
        if (j0 >= len) return false;                      // a shorter row has fewer spans
        if (lane != 0) return true;
        const int j1 = min(len, j0 + span_len);
        const int nq = enc ? p.beam : 1;
        const int first = enc ? p.enc_first[block] : p.self_first[block];
        const int pi = enc ? (p.enc_v_by_block ? 1 : p.enc_size[block]) : p.self_size[block];
        const int cap = enc ? p.cap_src : p.cap_tgt;
        const long long plane = enc ? p.mem_plane_bytes : p.self_plane_bytes;
        const long long panel = (((long long)id * p.H + h) * cap) * ROW_BYTES;
        const int nspans_max = enc ? p.enc_nspans : p.self_nspans;
        d->kind = enc ? 1 : 0; d->nq = nq; d->pi = pi; d->len = len; d->j0 = j0; d->j1 = j1;
        d->n_spans = (len + span_len - 1) / span_len; d->span = (int)span;
        d->has_new = (!enc && j1 == len) ? 1 : 0;
        d->row_id = enc ? row : p.n_enc_rows + row;
        d->part_stride = enc ? p.enc_part_stride : p.self_part_stride;
        d->part = p.part + (enc ? 0 : p.self_part_base) + ((long long)row * nspans_max + span) * (long long)d->part_stride;
        d->v_plane = plane;
        if (enc) {
            d->q = p.q_enc + ((((long long)block * p.n_sent + item) * nq) * p.H + h) * ROW_BYTES;
            d->q_stride = (long long)p.H * ROW_BYTES;
            d->Kp = p.memK + block * plane + panel;
            d->Vp = p.memV + (p.enc_v_by_block ? (int)block : first) * plane + panel;
            d->knew = nullptr; d->vnew = nullptr; d->vnew_stride = 0;
            d->S = p.S_enc ? p.S_enc + ((((long long)block * p.n_sent + item) * nq) * p.H + h) * p.ld_s : nullptr;
            d->S_qstride = (long long)p.H * p.ld_s;
            const int o_first = p.enc_v_by_block ? (int)block : first;
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
        return true;
    }

    // Makes the next item that is not skipped the one being issued.
    __device__ void next_item() {
        p_active = false;
        while (nx_item < p.n_items) {
            ItemDesc* d = &descs[p_n % kDescSlots];
            const bool ok = decode(nx_item, nx_id, nx_len, d);
            // shift the look-ahead: the item after becomes next (its metadata loads start now)
            nx_item = nn_item;
            fetch_meta(nx_item, &nx_id, &nx_len);
            nn_item = (nx_item < p.n_items) ? grab() : nx_item;
            if (ok) {
                __syncwarp();
                p_n += 1; p_active = true;
                p_q_done = 0; p_which = 0; p_j0 = d->j0; p_j1 = d->j1; p_pi = d->pi; p_s0 = p_j0;
                p_panel = d->Kp;
                return;
            }
        }
    }

    // Issues the copies of one tile of the item being issued, if any is left.
    __device__ void produce() {
        if (dead || !p_active) return;
        const ItemDesc& d = descs[(p_n - 1) % kDescSlots];
        const unsigned s = p_seq % kFusedStages;
        if (lane == 0) {
            const uint32_t dst = ring + s * kStageBytes;
            const uint32_t bar = bars + s * 8;
            if (!p_q_done) {
                mbar_expect_tx(bar, (uint32_t)(d.nq * ROW_BYTES));
                for (int qi = 0; qi < d.nq; ++qi) bulk_g2s(dst + qi * ROW_BYTES, d.q + qi * d.q_stride, ROW_BYTES, bar);
            } else {
                const int r = min(TR, p_j1 - p_s0);
                const bool with_new = d.has_new && (p_s0 + r == p_j1);
                const int r_cache = with_new ? r - 1 : r;
                mbar_expect_tx(bar, (uint32_t)(r * ROW_BYTES));
                if (r_cache > 0) bulk_g2s(dst, p_panel + (long long)p_s0 * ROW_BYTES, (uint32_t)(r_cache * ROW_BYTES), bar);
                if (with_new) {
                    const char* nsrc = p_which == 0 ? d.knew : d.vnew + (long long)(p_which - 1) * d.vnew_stride;
                    bulk_g2s(dst + r_cache * ROW_BYTES, nsrc, ROW_BYTES, bar);
                }
            }
        }
        p_seq += 1;
        if (!p_q_done) { p_q_done = 1; return; }
        p_s0 += TR;
        if (p_s0 >= p_j1) {
            p_which += 1; p_s0 = p_j0;
            if (p_which > p_pi) { next_item(); return; }
            p_panel = d.Vp + (long long)(p_which - 1) * d.v_plane;
        }
    }

    // Waits for the next tile in order; returns its stage or null after a timeout.
    __device__ __forceinline__ const char* acquire() {
        const unsigned s = c_seq % kFusedStages;
        const uint32_t bar = bars + s * 8, par = (c_seq / kFusedStages) & 1;
        if (!mbar_try_wait(bar, par)) {
            if (!mbar_wait_slow(bar, par)) {
                if (lane == 0 && atomicCAS(&p.err[0], 0, (int)SAN_ERR_TIMEOUT) == 0) { p.err[1] = TAG_STEP; p.err[2] = (int)c_seq; }
                dead = true;
                return nullptr;
            }
        }
        return ring_g + s * kStageBytes;
    }
    // Every lane is done with the tile: hand the stage back to the copy side.
    __device__ __forceinline__ void release() {
        // the tensor-core path writes into its tiles (chunk-permuting the newest row, zeroing a
        // ragged tail): order those writes ahead of the bulk copy that will reuse the stage
        if (sizeof(T) == 2) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        c_seq += 1;
        produce();
    }

    template <int NQ> __device__ bool process(const ItemDesc& d);
    template <int NQ> __device__ bool process_mma(const ItemDesc& d);
    template <int NQ> __device__ void combine(const ItemDesc& d);

    // bf16 tiles only.  A tile's last row may be this step's new row, copied in natural chunk
    // order from the caller's buffer: permute its chunks like a cached row (chunk c -> c ^ (pos & 7))
    // and write it to the cache at `dst_row`.  Rows [r, next multiple of 16) are zeroed when
    // `zero_tail` is set, so that a 16-row block never multiplies stale shared memory.
    __device__ __forceinline__ void fix_tile(const char* st, int r, bool with_new, char* dst_row, bool zero_tail) {
        if (with_new) {
            char* row = const_cast<char*>(st) + (r - 1) * 128;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (lane < 8) v = *reinterpret_cast<const uint4*>(row + lane * 16);
            __syncwarp();
            if (lane < 8) {
                const int pc = lane ^ ((r - 1) & 7);
                *reinterpret_cast<uint4*>(row + pc * 16) = v;
                *reinterpret_cast<uint4*>(dst_row + pc * 16) = v;
            }
        }
        if (zero_tail && (r & 15)) {
            const int r16 = (r + 15) & ~15;
            for (int j = r + (lane >> 3); j < r16; j += 4)
                *reinterpret_cast<uint4*>(const_cast<char*>(st) + j * 128 + (lane & 7) * 16) = make_uint4(0, 0, 0, 0);
        }
        __syncwarp();
    }

    // After a timeout: copies already issued may still land in this warp's stages, so give
    // each a last bounded chance to finish before the CTA's shared memory can go away.
    __device__ void drain() {
        while (c_seq != p_seq) {
            const unsigned s = c_seq % kFusedStages;
            const uint32_t par = (c_seq / kFusedStages) & 1;
            const long long t0 = clock64();
            while (!mbar_try_wait(bars + s * 8, par)) { if (clock64() - t0 > 200000000LL) break; }
            c_seq += 1;
        }
    }
};

template <typename T>
template <int NQ>
__device__ bool FusedWarp<T>::process(const ItemDesc& d) {
    constexpr int ZQ = kZFloats / NQ;          // score slots per query row
    constexpr int HDR = (2 * NQ + 3) / 4 * 4;  // (max, sum) per query ahead of a span's partial sums
    const int j0 = d.j0, n = d.j1 - d.j0, nq = d.nq, has_new = d.has_new, pi = d.pi;

    // ---- tile 0: the query rows, scaled into the log2 domain
    float2 q2[NQ][NP];
    {
        const char* st = acquire();
        if (!st) return false;
        const float sc = p.scale_log2e;
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) {
            if (qi < nq) {
                P::load(*reinterpret_cast<const uint4*>(st + qi * ROW_BYTES + c * 16), q2[qi]);
#pragma unroll
                for (int e = 0; e < NP; ++e) { q2[qi][e].x *= sc; q2[qi][e].y *= sc; }
            } else {
#pragma unroll
                for (int e = 0; e < NP; ++e) q2[qi][e] = make_float2(0.f, 0.f);
            }
        }
        release();
    }

    // ---- key tiles: scores into zs
    for (int s0 = 0; s0 < n; s0 += TR) {
        const char* st = acquire();
        if (!st) return false;
        const int r = min(TR, n - s0);
        const bool with_new = has_new && (s0 + r == n);
        for (int jb = 0; jb < r; jb += BLK) {
            uint4 kv[UN];
#pragma unroll
            for (int u = 0; u < UN; ++u) {
                const int j = jb + u * RPW + g;
                kv[u] = (j < r) ? *reinterpret_cast<const uint4*>(st + j * ROW_BYTES + c * 16) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < UN; ++u) {
                const int j = jb + u * RPW + g;
                float2 k2[NP];
                P::load(kv[u], k2);
#pragma unroll
                for (int qi = 0; qi < NQ; ++qi) {
                    float2 a = make_float2(0.f, 0.f);
#pragma unroll
                    for (int e = 0; e < NP; ++e) a = __ffma2_rn(q2[qi][e], k2[e], a);
                    float dot = a.x + a.y;
#pragma unroll
                    for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                    if (c == 0 && j < r) zs[qi * ZQ + s0 + j] = dot;
                }
                // the newest key row goes into the cache from here
                if (with_new && j == r - 1)
                    *reinterpret_cast<uint4*>(const_cast<char*>(d.Kp) + (long long)(d.len - 1) * ROW_BYTES + c * 16) = kv[u];
            }
        }
        release();
    }

    // ---- softmax over the span (log2 domain)
    float part_m[NQ], part_l[NQ];
    const int n_spans = d.n_spans;
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
            float* Srow = d.S ? d.S + qi * d.S_qstride + j0 : nullptr;
            if (n_spans == 1) {
                const float inv = 1.0f / s;
                for (int jj = lane; jj < n; jj += 32) {
                    const float w = zs[qi * ZQ + jj] * inv;
                    zs[qi * ZQ + jj] = w;
                    if (Srow) Srow[jj] = w;
                }
            } else if (Srow) {
                for (int jj = lane; jj < n; jj += 32) Srow[jj] = zs[qi * ZQ + jj];
            }
        }
    }
    __syncwarp();

    // ---- value tiles, layer by layer (score rows of absent queries hold zeros)
    for (int l = 0; l < pi; ++l) {
        float2 acc[NQ][NP];
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi)
#pragma unroll
            for (int e = 0; e < NP; ++e) acc[qi][e] = make_float2(0.f, 0.f);
        for (int s0 = 0; s0 < n; s0 += TR) {
            const char* st = acquire();
            if (!st) return false;
            const int r = min(TR, n - s0);
            const bool with_new = has_new && (s0 + r == n);
            for (int jb = 0; jb < r; jb += BLK) {
                uint4 vv[UN];
#pragma unroll
                for (int u = 0; u < UN; ++u) {
                    const int j = jb + u * RPW + g;
                    vv[u] = (j < r) ? *reinterpret_cast<const uint4*>(st + j * ROW_BYTES + c * 16) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int u = 0; u < UN; ++u) {
                    const int j = jb + u * RPW + g;
                    if (j < r) {
                        float2 v2[NP];
                        P::load(vv[u], v2);
#pragma unroll
                        for (int qi = 0; qi < NQ; ++qi) {
                            const float s = zs[qi * ZQ + s0 + j];
                            const float2 ss = make_float2(s, s);
#pragma unroll
                            for (int e = 0; e < NP; ++e) acc[qi][e] = __ffma2_rn(ss, v2[e], acc[qi][e]);
                        }
                        if (with_new && j == r - 1)
                            *reinterpret_cast<uint4*>(const_cast<char*>(d.Vp) + (long long)l * d.v_plane +
                                                      (long long)(d.len - 1) * ROW_BYTES + c * 16) = vv[u];
                    }
                }
            }
            release();
        }
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi)
#pragma unroll
            for (int e = 0; e < NP; ++e)
#pragma unroll
                for (int o = LPR; o < 32; o <<= 1) {
                    acc[qi][e].x += __shfl_xor_sync(0xffffffffu, acc[qi][e].x, o);
                    acc[qi][e].y += __shfl_xor_sync(0xffffffffu, acc[qi][e].y, o);
                }
        if (g == 0) {
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) {
                if (qi < nq) {
                    if (n_spans == 1) {
                        *reinterpret_cast<uint4*>(d.O + l * d.O_lstride + qi * d.O_qstride + c * 16) = P::store(acc[qi]);
                    } else {
                        float2* pp = reinterpret_cast<float2*>(d.part + HDR + ((long long)l * NQ + qi) * kDh + c * VEC);
#pragma unroll
                        for (int e = 0; e < NP; ++e) pp[e] = acc[qi][e];
                    }
                }
            }
        }
    }
    if (n_spans == 1) return true;

    // ---- split row: park (max, sum); the last span to arrive combines all of them
    if (lane == 0) {
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) { d.part[qi] = part_m[qi]; d.part[NQ + qi] = part_l[qi]; }
    }
    __threadfence();
    __syncwarp();
    int t = 0;
    if (lane == 0) t = atomicAdd(p.tickets + d.row_id, 1);
    t = __shfl_sync(0xffffffffu, t, 0);
    if (t == n_spans - 1) combine<NQ>(d);
    return true;
}

// bf16 items on the tensor cores (mma.sync m16n8k16, float32 accumulate).  Neither product
// is a dense GEMM: the tensor cores are used because one 16-row block of a tile then costs
// a handful of instructions (4 ldmatrix + 4 mma for the scores, 4 ldmatrix + 16 mma for one
// layer's S.V) instead of a hundred or more unpack/FMA/shuffle instructions, and the step
// is bound by instruction issue, not by tensor throughput.
//   scores:  D[16 positions x 8 queries] = K_tile[16 x 64] . q^T          (queries padded to 8)
//   apply:   D[16 queries x 8 dims]     += S[16 x 16 positions] . V_tile   (eight dim tiles)
// S is split into a bf16 high part and a bf16 remainder (two MMAs) so that the weights keep
// about 16 bits; products and sums are float32.
template <typename T>
template <int NQ>
__device__ bool FusedWarp<T>::process_mma(const ItemDesc& d) {
    static_assert(sizeof(T) == 2, "tensor-core path is for bf16 rows");
    constexpr int ZQ = kZFloats / NQ;
    constexpr int HDR = (2 * NQ + 3) / 4 * 4;
    const int j0 = d.j0, n = d.j1 - d.j0, nq = d.nq, has_new = d.has_new, pi = d.pi;
    const int tig = lane & 3, gid = lane >> 2;                 // mma fragment coordinates
    const int lrow = (lane & 7) + ((lane >> 3) & 1) * 8;        // ldmatrix: row of the 16-row block this lane addresses
    const int lx = lane & 7, lsel = lane >> 4;                  // its chunk permutation key and chunk of the pair

    // ---- tile 0: the query rows as B fragments (k = dims, n = query), natural chunk order
    uint32_t qb[4][2];
    {
        const char* st = acquire();
        if (!st) return false;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            qb[ks][0] = 0u; qb[ks][1] = 0u;
            if (gid < nq) {
                qb[ks][0] = *reinterpret_cast<const uint32_t*>(st + gid * 128 + (16 * ks + 2 * tig) * 2);
                qb[ks][1] = *reinterpret_cast<const uint32_t*>(st + gid * 128 + (16 * ks + 8 + 2 * tig) * 2);
            }
        }
        release();
    }

    // ---- key tiles: scores into zs (log2 domain)
    const float sc = p.scale_log2e;
    for (int s0 = 0; s0 < n; s0 += TR) {
        const char* st = acquire();
        if (!st) return false;
        const int r = min(TR, n - s0);
        fix_tile(st, r, has_new && (s0 + r == n), const_cast<char*>(d.Kp) + (long long)(d.len - 1) * 128, false);
        const uint32_t st_s = ring + (uint32_t)(st - ring_g);
        for (int b0 = 0; b0 < r; b0 += 16) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                uint32_t a[4];
                ldsm_x4(st_s + (b0 + lrow) * 128 + (((2 * ks + lsel) ^ lx) << 4), a);
                mma_bf16(acc, a[0], a[1], a[2], a[3], qb[ks][0], qb[ks][1]);
            }
            // acc[0], acc[1]: position b0+gid, queries 2tig, 2tig+1; acc[2], acc[3]: position b0+gid+8
            const int p0 = b0 + gid, p1 = b0 + gid + 8;
            if (2 * tig < NQ) {
                if (p0 < r) zs[(2 * tig) * ZQ + s0 + p0] = acc[0] * sc;
                if (p1 < r) zs[(2 * tig) * ZQ + s0 + p1] = acc[2] * sc;
            }
            if (2 * tig + 1 < NQ) {
                if (p0 < r) zs[(2 * tig + 1) * ZQ + s0 + p0] = acc[1] * sc;
                if (p1 < r) zs[(2 * tig + 1) * ZQ + s0 + p1] = acc[3] * sc;
            }
        }
        release();
    }
    __syncwarp();

    // ---- softmax over the span (log2 domain)
    float part_m[NQ], part_l[NQ];
    const int n_spans = d.n_spans;
    const int n16 = (n + 15) & ~15;
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
            float* Srow = d.S ? d.S + qi * d.S_qstride + j0 : nullptr;
            if (n_spans == 1) {
                const float inv = 1.0f / s;
                for (int jj = lane; jj < n; jj += 32) {
                    const float w = zs[qi * ZQ + jj] * inv;
                    zs[qi * ZQ + jj] = w;
                    if (Srow) Srow[jj] = w;
                }
            } else if (Srow) {
                for (int jj = lane; jj < n; jj += 32) Srow[jj] = zs[qi * ZQ + jj];
            }
        }
        // weights beyond the span's end (up to the next multiple of 16) must be exactly zero
        for (int jj = n + lane; jj < n16; jj += 32) zs[qi * ZQ + jj] = 0.f;
    }
    __syncwarp();

    // ---- value tiles, layer by layer
    for (int l = 0; l < pi; ++l) {
        float acc[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[nt][e] = 0.f;
        for (int s0 = 0; s0 < n; s0 += TR) {
            const char* st = acquire();
            if (!st) return false;
            const int r = min(TR, n - s0);
            fix_tile(st, r, has_new && (s0 + r == n),
                     const_cast<char*>(d.Vp) + (long long)l * d.v_plane + (long long)(d.len - 1) * 128, true);
            const uint32_t st_s = ring + (uint32_t)(st - ring_g);
            for (int b0 = 0; b0 < r; b0 += 16) {
                // A = weights of query gid at positions b0 + {2tig, 2tig+1, 2tig+8, 2tig+9}: high part + remainder
                uint32_t ah0 = 0u, ah2 = 0u, al0 = 0u, al2 = 0u;
                if (gid < NQ) {
                    const float2 w0 = *reinterpret_cast<const float2*>(zs + gid * ZQ + s0 + b0 + 2 * tig);
                    const float2 w1 = *reinterpret_cast<const float2*>(zs + gid * ZQ + s0 + b0 + 2 * tig + 8);
                    ah0 = pack_bf16x2(w0.x, w0.y); ah2 = pack_bf16x2(w1.x, w1.y);
                    al0 = pack_bf16x2(w0.x - __uint_as_float(ah0 << 16), w0.y - __uint_as_float(ah0 & 0xffff0000u));
                    al2 = pack_bf16x2(w1.x - __uint_as_float(ah2 << 16), w1.y - __uint_as_float(ah2 & 0xffff0000u));
                }
#pragma unroll
                for (int np = 0; np < 4; ++np) {
                    uint32_t b[4];
                    ldsm_x4_t(st_s + (b0 + lrow) * 128 + (((2 * np + lsel) ^ lx) << 4), b);
                    mma_bf16(acc[2 * np], ah0, 0u, ah2, 0u, b[0], b[1]);
                    mma_bf16(acc[2 * np + 1], ah0, 0u, ah2, 0u, b[2], b[3]);
                    mma_bf16(acc[2 * np], al0, 0u, al2, 0u, b[0], b[1]);
                    mma_bf16(acc[2 * np + 1], al0, 0u, al2, 0u, b[2], b[3]);
                }
            }
            release();
        }
        // acc[nt][0], acc[nt][1]: query gid, dims 8nt + 2tig, +1
        if (gid < nq) {
            if (n_spans == 1) {
                char* op = d.O + l * d.O_lstride + gid * d.O_qstride + 4 * tig;
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) *reinterpret_cast<uint32_t*>(op + 16 * nt) = pack_bf16x2(acc[nt][0], acc[nt][1]);
            } else {
                float* pp = d.part + HDR + ((long long)l * NQ + gid) * kDh + 2 * tig;
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) *reinterpret_cast<float2*>(pp + 8 * nt) = make_float2(acc[nt][0], acc[nt][1]);
            }
        }
    }
    if (n_spans == 1) return true;

    if (lane == 0) {
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) { d.part[qi] = part_m[qi]; d.part[NQ + qi] = part_l[qi]; }
    }
    __threadfence();
    __syncwarp();
    int t = 0;
    if (lane == 0) t = atomicAdd(p.tickets + d.row_id, 1);
    t = __shfl_sync(0xffffffffu, t, 0);
    if (t == n_spans - 1) combine<NQ>(d);
    return true;
}

// The last span of a split row: softmax weights across spans, then S and every layer's O.
template <typename T>
template <int NQ>
__device__ void FusedWarp<T>::combine(const ItemDesc& d) {
    constexpr int HDR = (2 * NQ + 3) / 4 * 4;
    __threadfence();
    const int n_spans = d.n_spans, nq = d.nq, stride = d.part_stride;
    const float* row_part = d.part - (long long)d.span * stride;
    const int span_len = d.kind ? p.enc_span : p.self_span;
    // zs[sp * NQ + qi] = exp2(m_sp - M) / total  (zs is free: every layer of this span is done)
    __syncwarp();
    for (int qi = 0; qi < NQ; ++qi) {
        float m = -INFINITY, l = 0.f;
        if (lane < n_spans && qi < nq) { m = __ldcg(row_part + (long long)lane * stride + qi); l = __ldcg(row_part + (long long)lane * stride + NQ + qi); }
        const float M = warp_max(m);
        const float wl = (lane < n_spans && qi < nq) ? l * exp2f(m - M) : 0.f;
        const float tot = warp_sum(wl);
        if (lane < n_spans) zs[lane * NQ + qi] = (qi < nq) ? exp2f(m - M) / tot : 0.f;
    }
    __syncwarp();
    if (d.S) {
        for (int qi = 0; qi < nq; ++qi) {
            float* Srow = d.S + qi * d.S_qstride;
            for (int j = lane; j < d.len; j += 32) Srow[j] = __ldcg(Srow + j) * zs[(j / span_len) * NQ + qi];
        }
    }
    // every layer's output: E = pi*NQ*64 floats per span, four per lane per pass
    const int E = d.pi * NQ * kDh;
    for (int e0 = lane * 4; e0 < E; e0 += 128) {
        const int qi = (e0 / kDh) % NQ;
        if (qi >= nq) continue;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        const float* src = row_part + HDR + e0;
        int sp = 0;
        for (; sp + 4 <= n_spans; sp += 4) {
            float4 x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) x[u] = __ldcg(reinterpret_cast<const float4*>(src + (long long)(sp + u) * stride));
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float f = zs[(sp + u) * NQ + qi];
                a.x = fmaf(f, x[u].x, a.x); a.y = fmaf(f, x[u].y, a.y); a.z = fmaf(f, x[u].z, a.z); a.w = fmaf(f, x[u].w, a.w);
            }
        }
        for (; sp < n_spans; ++sp) {
            const float4 x = __ldcg(reinterpret_cast<const float4*>(src + (long long)sp * stride));
            const float f = zs[sp * NQ + qi];
            a.x = fmaf(f, x.x, a.x); a.y = fmaf(f, x.y, a.y); a.z = fmaf(f, x.z, a.z); a.w = fmaf(f, x.w, a.w);
        }
        const int ly = e0 / (NQ * kDh), col = e0 % kDh;
        char* op = d.O + ly * d.O_lstride + qi * d.O_qstride + col * (int)sizeof(T);
        if (sizeof(T) == 2) {
            __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(a.z, a.w);
            uint2 r; r.x = *reinterpret_cast<uint32_t*>(&lo); r.y = *reinterpret_cast<uint32_t*>(&hi);
            *reinterpret_cast<uint2*>(op) = r;
        } else {
            *reinterpret_cast<float4*>(op) = a;
        }
    }
    if (lane == 0) p.tickets[d.row_id] = 0;
}

constexpr size_t fused_smem_bytes() {
    return (size_t)kFusedWarps * (kFusedStages * kStageBytes + kZFloats * sizeof(float) + kDescSlots * sizeof(ItemDesc) +
                                  kFusedStages * sizeof(uint64_t)) + 128;
}

template <typename T, int NQE>
__global__ void __launch_bounds__(kFusedWarps * 32, 1) decode_step_kernel(const __grid_constant__ StepParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ unsigned cta_next;
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
    if (threadIdx.x == 0) cta_next = kFusedWarps;   // slots 0..warps-1 are the warps' first items
    __syncthreads();
    FusedWarp<T> w(p);
    char* base = reinterpret_cast<char*>(smem);
    w.ring_g = base + (size_t)warp * kFusedStages * kStageBytes;
    w.ring = smem_u32(w.ring_g);
    char* after = base + (size_t)kFusedWarps * kFusedStages * kStageBytes;
    w.zs = reinterpret_cast<float*>(after) + (size_t)warp * kZFloats;
    after += (size_t)kFusedWarps * kZFloats * sizeof(float);
    w.descs = reinterpret_cast<ItemDesc*>(after) + (size_t)warp * kDescSlots;
    after += (size_t)kFusedWarps * kDescSlots * sizeof(ItemDesc);
    uint64_t* bars_g = reinterpret_cast<uint64_t*>(after) + (size_t)warp * kFusedStages;
    w.bars = smem_u32(bars_g);
    w.cta_next = &cta_next;
    w.lane = lane; w.g = lane / RowGeom<T>::LPR; w.c = lane % RowGeom<T>::LPR;
    w.p_seq = 0; w.p_n = 0; w.c_seq = 0; w.c_n = 0; w.dead = false; w.p_active = false;
    if (lane == 0) {
        for (int s = 0; s < kFusedStages; ++s) mbar_init(bars_g + s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    w.nx_item = w.item_of_slot((unsigned)warp);
    w.fetch_meta(w.nx_item, &w.nx_id, &w.nx_len);
    w.nn_item = (w.nx_item < p.n_items) ? w.grab() : w.nx_item;
    w.next_item();
    for (int s = 0; s < kFusedStages; ++s) w.produce();
    while (w.c_n < w.p_n && !w.dead) {
        const ItemDesc& d = w.descs[w.c_n % kDescSlots];
        if constexpr (sizeof(T) == 2) {
            if (d.kind) w.template process_mma<NQE>(d); else w.template process_mma<1>(d);
        } else {
            if (d.kind) w.template process<NQE>(d); else w.template process<1>(d);
        }
        w.c_n += 1;
    }
    if (w.dead) w.drain();
}

}  // namespace san
