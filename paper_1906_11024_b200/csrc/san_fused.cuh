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
// Two stages per warp keep the copies ahead of the arithmetic as well as three did (measured),
// and leave the shared memory for longer spans: a row of up to kZFloats / NQ positions needs
// no partial sums and no combine.
constexpr int kFusedStages = 2;
constexpr int kZFloats = 1024;      // scores a warp keeps on chip: span <= kZFloats / NQ
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

// Everything that differs between the two attention kinds, filled by the host.
struct KindParams {
    const char* q; const char* K; const char* V;      // queries; key / value plane 0 of the kind
    const char* knew; const char* vnew;               // this step's rows (self only, else null)
    float* S; char* O;                                 // S may be null
    const int* ids; const int* lens;                   // lens: source lengths (enc-dec) or write positions (self)
    long long plane_bytes;                             // between cache planes
    long long layer_bytes;                             // between layers in O and v_new / blocks in k_new: n_it*nq*H*row bytes
    long long S_ld;                                    // floats between S rows
    long long part_base;                               // float offset of the kind's partial sums
    unsigned panel_bytes;                              // capacity * row bytes: one (id, head) panel
    unsigned n_it, nq, len_bias, max_ids, bound;       // items, query rows per item in this launch, 1 if lens holds positions, limits
    unsigned q_first, q_total;                         // first of those rows among the q_total rows an item has in q, S and O
    unsigned span, nspans, part_stride, v_by_block, row_base;
    unsigned lg_size, n_lg;                            // layers per item (a block is cut into groups), groups per block at most
    unsigned hpi;                                      // heads per item (1 unless the short-rows kernel takes several side by side); div_h divides by H / hpi
    FastDiv div_span, div_lg, div_h, div_item;
    unsigned char first[SAN_MAX_LAYERS], size[SAN_MAX_LAYERS];   // per block
};

struct StepParams {
    KindParams k[2];                                   // [0] decoder self-attention, [1] encoder-decoder attention
    unsigned n_enc_items, n_items;                     // enc-dec items come first in the list
    int H;
    float* part; int* tickets; int* err;
    float scale_log2e;
    // AAN in place of self-attention (absent when x_aan == null)
    const char* x_aan; const int* t_aan; const int* aan_ids; float* aan_sum; char* aan_out;
    int n_aan_layers, n_aan_seqs, aan_max_seqs, aan_max_t;
};

// A decoded work item, kept in shared memory between the copy side and the math side.
struct ItemDesc {
    const char* q;                            // query row 0
    const char* srcK;                         // key panel, first row of the span
    const char* srcV;                         // value panel of the item's first layer, first row of the span
    const char* knew; const char* vnew;       // newest rows (self only): key row; value row of the item's first layer
    float* S;                                 // S row of query 0 at the span's first position (null: not stored)
    char* O;                                  // output of (first layer, query 0)
    float* part;                              // partial sums of this (row, span)
    unsigned row_id;                          // ticket index of the row
    int n;                                    // positions in the span
    int len;                                  // positions in the whole row
    int kind, nq, pi, n_spans, span;
    int has_new;                              // the span's last position is this step's row, not yet in the cache
    int lead;                                 // this item also stores the key row of the step
    int heads;                                // heads it covers, from the one its pointers name
};

// The kernel's dynamic shared memory.  Everything a warp keeps there is addressed by a 32-bit
// byte offset into this array, so that the compiler emits shared-space loads and stores with
// 32-bit address arithmetic instead of generic 64-bit pointers.
extern __shared__ __align__(128) unsigned char san_smem[];
template <typename U> __device__ __forceinline__ U* sp(uint32_t off) { return reinterpret_cast<U*>(san_smem + off); }

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
// try_wait that lets the hardware keep the thread suspended for a while (it returns as soon as
// the phase completes), so that a waiting warp does not use issue slots.  Measured on B200: a
// hint of 1,000,000 suspends for about 1000 cycles; without a hint the instruction returns at once.
__device__ __forceinline__ bool mbar_try_wait_hint(uint32_t bar, uint32_t parity, uint32_t hint) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(hint) : "memory");
    return ok != 0;
}
// Polls the barrier up to `tries` times, each try suspending the thread for a while; true once the
// phase is complete.  A suspended thread is woken whenever any barrier of the CTA completes, far more
// often than its own does, so the loop is kept to four instructions a turn.
__device__ __forceinline__ bool mbar_poll(uint32_t bar, uint32_t parity, uint32_t hint, uint32_t tries) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        ".reg .u32 n;\n"
        "mov.u32 n, %4;\n"
        "POLL:\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
        "@p bra DONE;\n"
        "sub.u32 n, n, 1;\n"
        "setp.ne.u32 p, n, 0;\n"
        "@p bra POLL;\n"
        "setp.ne.u32 p, n, 0;\n"
        "DONE:\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(hint), "r"(tries) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after about a second and reports it; never spins for ever.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity) {
    const long long t0 = clock64();
    do {
        if (mbar_poll(bar, parity, 2000000u, 4096u)) return true;
    } while (clock64() - t0 < 2000000000LL);
    return false;
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
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
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

// ------------------------------------------------------------------------------ decoding
// Item `it` of the list ([enc-dec items][self items]; within a kind (((block, item), head),
// span)) into *d.  Returns false if the item is to be skipped (a failed device check, which
// is recorded, or a span beyond the row's length).  Called by one thread per item: a CTA
// decodes its whole share of the list side by side before any arithmetic starts.
template <int ROW_BYTES>
__device__ bool decode_item(const StepParams& p, unsigned it, ItemDesc* d) {
    const int enc = it < p.n_enc_items;
    const KindParams& kp = p.k[enc];
    unsigned row, span, bi, h, block, item, rl, lg;
    kp.div_span.divmod(enc ? it : it - p.n_enc_items, &rl, &span);    // rl = (row, layer group)
    kp.div_lg.divmod(rl, &row, &lg);
    kp.div_h.divmod(row, &bi, &h);
    h *= kp.hpi;
    kp.div_item.divmod(bi, &block, &item);
    const int id = kp.ids[item], len = kp.lens[item] + (int)kp.len_bias;
    const bool reporter = (span == 0 && lg == 0 && h == 0 && block == 0);
    if ((unsigned)id >= kp.max_ids) { if (reporter) record_error(p.err, TAG_STEP, (int)item, id, (int)kp.max_ids); return false; }
    if (len < 1 || len > (int)kp.bound) { if (reporter) record_error(p.err, TAG_STEP, (int)item, len, (int)kp.bound); return false; }
    const int j0 = (int)(span * kp.span);
    if (j0 >= len) return false;                      // a shorter row has fewer spans
    const unsigned size = kp.v_by_block ? 1u : kp.size[block];
    const unsigned l0 = lg * kp.lg_size;              // first layer of the group, relative to the block
    if (l0 >= size) return false;                     // a smaller block has fewer layer groups
    const unsigned H = (unsigned)p.H;
    const int j1 = min(len, j0 + (int)kp.span);
    const unsigned first = kp.first[block] + l0;      // every group recomputes S from the block's keys
    const unsigned vplane = (kp.v_by_block ? block : kp.first[block]) + l0;
    const unsigned qrow = ((block * kp.n_it + item) * kp.q_total + kp.q_first) * H + h;   // row of the launch's query 0 in q and S
    const unsigned long long panel = (unsigned long long)((unsigned)id * H + h) * kp.panel_bytes;
    d->kind = enc; d->nq = (int)kp.nq; d->pi = (int)min(kp.lg_size, size - l0);
    d->len = len; d->n = j1 - j0;
    d->n_spans = (len + (int)kp.span - 1) / (int)kp.span; d->span = (int)span;
    d->has_new = (kp.knew != nullptr && j1 == len) ? 1 : 0;
    d->heads = (int)kp.hpi;
    d->lead = (lg == 0) ? 1 : 0;                      // the group that also stores S and this step's key row
    d->row_id = kp.row_base + rl;
    d->part = p.part + kp.part_base + (unsigned long long)(rl * kp.nspans + span) * kp.part_stride;
    d->q = kp.q + (unsigned long long)qrow * ROW_BYTES;
    d->S = (kp.S && lg == 0) ? kp.S + (unsigned long long)qrow * (unsigned long long)kp.S_ld + j0 : nullptr;
    d->srcK = kp.K + (unsigned long long)block * (unsigned long long)kp.plane_bytes + panel + (unsigned)j0 * ROW_BYTES;
    d->srcV = kp.V + (unsigned long long)vplane * (unsigned long long)kp.plane_bytes + panel + (unsigned)j0 * ROW_BYTES;
    d->O = kp.O + (unsigned long long)vplane * (unsigned long long)kp.layer_bytes +
           (unsigned long long)((item * kp.q_total + kp.q_first) * H + h) * ROW_BYTES;
    const unsigned long long in_row = (unsigned long long)(item * H + h) * ROW_BYTES;   // self: nq == 1
    d->knew = kp.knew ? kp.knew + (unsigned long long)block * (unsigned long long)kp.layer_bytes + in_row : nullptr;
    d->vnew = kp.vnew ? kp.vnew + (unsigned long long)first * (unsigned long long)kp.layer_bytes + in_row : nullptr;
    return true;
}

// ------------------------------------------------------------------------------ the warp
template <typename T, int NQ>
__device__ void combine_spans(const StepParams& p, const ItemDesc& d, uint32_t zs_off, int lane);

template <typename T>
struct FusedWarp {
    using G = RowGeom<T>;
    using F = FusedGeom<T>;
    using P = Pairs<T>;
    static constexpr int VEC = G::VEC, LPR = G::LPR, RPW = 32 / LPR, ROW_BYTES = F::ROW_BYTES, TR = F::TR;
    static constexpr int QROW = TR - 8;      // the first key tile of an item holds key rows [0, QROW) and the
                                             // query rows from row QROW on (at most 8 of them)
    static constexpr int NP = P::N;          // float pairs per 16 bytes
    static constexpr int BLK = 8;            // rows per inner block
    static constexpr int UN = BLK / RPW;     // loads per lane per block

    const StepParams& p;
    uint32_t sm_base;             // shared-space address of san_smem (for PTX operands: address = sm_base + offset)
    uint32_t ring, bars;          // offsets of this warp's stages and of their barriers
    uint32_t zs_off;              // offset of its kZFloats score slots
    uint32_t descs_off;           // offset of the CTA's decoded items
    uint32_t zero_row;            // shared-space address of 128 zero bytes
    unsigned* q_next;             // shared counter: next of them to hand out
    unsigned n_valid;             // how many there are
    int lane;
    // copy side: the item whose tiles are being issued, and the one after (taken ahead)
    bool p_active;
    bool p_first;                 // the next tile is the item's first key tile
    unsigned p_idx, nx_idx, p_stage;
    int p_which;                  // panel being issued: 0 = keys, l + 1 = values of the item's layer l
    int p_pi, p_n, p_left, p_has_new, p_nq, p_kind;
    const char* p_src;            // next rows of the panel
    const char* p_new;            // this step's row of the panel (self only)
    // math side
    unsigned c_stage, c_par;
    unsigned long long fifo;      // items whose tiles are (being) issued and whose arithmetic is still to do,
    int fifo_n;                   // oldest in the low byte (item indices are below kCtaItems <= 255)
    bool dead;                    // a wait ran out: leave

    __device__ FusedWarp(const StepParams& pp) : p(pp) {}

    __device__ __forceinline__ const ItemDesc& desc(unsigned idx) const {
        return *sp<ItemDesc>(descs_off + idx * (uint32_t)sizeof(ItemDesc));
    }

    __device__ __forceinline__ unsigned grab() {
        unsigned k = 0;
        if (lane == 0) k = atomicAdd(q_next, 1u);
        return __shfl_sync(0xffffffffu, k, 0);
    }

    // The copy side moves on to the item taken ahead, and takes the one after.
    __device__ __forceinline__ void next_item() {
        p_idx = nx_idx;
        p_active = p_idx < n_valid;
        if (!p_active) return;
        fifo |= (unsigned long long)p_idx << (8 * fifo_n);
        fifo_n += 1;
        nx_idx = grab();
        const ItemDesc& d = desc(p_idx);
        p_which = 0; p_first = true; p_pi = d.pi; p_n = d.n; p_left = p_n; p_has_new = d.has_new;
        p_nq = d.nq; p_kind = d.kind;
        p_src = d.srcK; p_new = d.knew;
    }

    // Issues the copies of one tile of the item being issued, if any is left.  The first key
    // tile of an item has room for QROW key rows and carries the query rows behind them.
    __device__ __forceinline__ void produce() {
        if (!p_active) return;
        if (!p_first && p_left > TR) {      // a whole tile from the middle of a panel: nothing else to decide
            if (lane == 0) {
                const uint32_t bar = sm_base + bars + p_stage * 8;
                mbar_expect_tx(bar, (uint32_t)kStageBytes);
                bulk_g2s(sm_base + ring + p_stage * kStageBytes, p_src, (uint32_t)kStageBytes, bar);
            }
            p_stage = (p_stage + 1 == (unsigned)kFusedStages) ? 0 : p_stage + 1;
            p_left -= TR;
            p_src += kStageBytes;
            return;
        }
        const int r = min(p_first ? QROW : TR, p_left);
        const bool with_new = p_has_new && (r == p_left);      // this step's row closes the panel
        const uint32_t cache_bytes = (uint32_t)(r - (with_new ? 1 : 0)) * ROW_BYTES;
        if (lane == 0) {
            const uint32_t dst = sm_base + ring + p_stage * kStageBytes;
            const uint32_t bar = sm_base + bars + p_stage * 8;
            mbar_expect_tx(bar, (uint32_t)(r + (p_first ? p_nq : 0)) * ROW_BYTES);
            if (cache_bytes) bulk_g2s(dst, p_src, cache_bytes, bar);
            if (with_new) bulk_g2s(dst + cache_bytes, p_new, ROW_BYTES, bar);
            if (p_first) {      // the query rows ride behind the first key tile
                const char* q = desc(p_idx).q;
                const unsigned q_stride = (unsigned)p.H * ROW_BYTES;
#pragma unroll 1
                for (int qi = 0; qi < p_nq; ++qi, q += q_stride) bulk_g2s(dst + (QROW + qi) * ROW_BYTES, q, ROW_BYTES, bar);
            }
        }
        p_first = false;
        p_stage = (p_stage + 1 == (unsigned)kFusedStages) ? 0 : p_stage + 1;
        p_left -= r;
        p_src += (uint32_t)r * ROW_BYTES;
        if (p_left <= 0) {
            if (p_which == p_pi) { next_item(); return; }
            if (p_which == 0) {                                 // on to the value panel of the item's first layer
                const ItemDesc& d = desc(p_idx);
                p_src = d.srcV; p_new = d.vnew;
            } else {                                            // the same rows of the next layer's plane
                p_src += p.k[p_kind].plane_bytes - (long long)((uint32_t)p_n * ROW_BYTES);
                p_new += p.k[p_kind].layer_bytes;
            }
            p_which += 1;
            p_left = p_n;
        }
    }

    // Waits for the next tile in order; returns the offset of its stage, or kNoTile after a timeout.
    static constexpr uint32_t kNoTile = 0xffffffffu;
    __device__ __forceinline__ uint32_t acquire() {
        const uint32_t bar = sm_base + bars + c_stage * 8;
        if (!mbar_try_wait(bar, c_par)) {
            if (!mbar_wait_slow(bar, c_par)) {
                if (lane == 0 && atomicCAS(&p.err[0], 0, (int)SAN_ERR_TIMEOUT) == 0) { p.err[1] = TAG_STEP; p.err[2] = (int)c_stage; }
                dead = true;
                return kNoTile;
            }
        }
        return ring + c_stage * kStageBytes;
    }
    // Every lane is done with the tile (tiles are only ever read): its stage takes the next
    // tile to be issued.
    __device__ __forceinline__ void release() {
        __syncwarp();
        if (++c_stage == (unsigned)kFusedStages) { c_stage = 0; c_par ^= 1u; }
        produce();
    }

    template <int NQ> __device__ bool process(const ItemDesc& d);
    template <int NQ> __device__ bool process_mma(const ItemDesc& d);
    template <int NQ, bool PACK> __device__ __forceinline__ void softmax_span(const ItemDesc& d, int n, int n_pad);
};

// Where the bf16 high part of position `pos` goes in a packed score row, as a 16-bit index
// (the remainder sits 4 further): see softmax_span.
__device__ __forceinline__ int packed_slot(int pos) {
    const int jp = (pos >> 1) & 7;       // pair of positions within the block of 16
    return (((pos >> 4) << 4) + ((jp & 3) << 2) + (jp >> 2)) * 2 + (pos & 1);
}

// Softmax of the n scores of a span held in zs (log2 domain), per query row.  A span that is
// the whole row produces normalised weights and writes them to S; otherwise it produces
// exp2(z - max) and parks (max, sum) in the span's partial-sum record for the combine.  With PACK == false the weights are
// left in zs as floats (entries n .. n_pad zeroed).  With PACK == true (tensor-core path) they
// are left as bf16 pairs, split into a bf16 high part and a bf16 remainder (w - high), zero
// beyond n up to n_pad, in the order the MMA's B fragments want them: the 16 positions of a
// block take 16 words; thread-in-group t owns words 4t .. 4t+3 = high parts of positions
// (2t, 2t+1), high parts of (2t+8, 2t+9), remainders of (2t, 2t+1), remainders of (2t+8, 2t+9).
template <typename T>
template <int NQ, bool PACK>
__device__ __forceinline__ void FusedWarp<T>::softmax_span(const ItemDesc& d, int n, int n_pad) {
    constexpr int ZQ = kZFloats / NQ;
    const int nq = d.nq, n_spans = d.n_spans;
    const long long S_qstride = (long long)p.H * p.k[d.kind].S_ld;
    if (n <= 64) {
        // At most two scores per lane and no loops; the query rows go through the reductions side
        // by side, so that their shuffles overlap.  Rows of absent queries (padding up to NQ) hold
        // finite scores of a repeated query row: they are carried along and never stored.
        const bool two = n > 32;                       // warp-uniform
        const bool in0 = lane < n, in1 = lane + 32 < n;
        float z0[NQ], z1[NQ], m[NQ], sum[NQ];
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) {
            const float* zq = sp<float>(zs_off + qi * ZQ * 4);
            z0[qi] = in0 ? zq[lane] : -INFINITY;
            z1[qi] = (two && in1) ? zq[lane + 32] : -INFINITY;
            m[qi] = fmaxf(z0[qi], z1[qi]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) m[qi] = fmaxf(m[qi], __shfl_xor_sync(0xffffffffu, m[qi], o));
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) {
            z0[qi] = exp2f(z0[qi] - m[qi]);             // exp2(-inf) = 0 for the lanes beyond n
            z1[qi] = exp2f(z1[qi] - m[qi]);
            sum[qi] = z0[qi] + z1[qi];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) sum[qi] += __shfl_xor_sync(0xffffffffu, sum[qi], o);
        __syncwarp();                                   // every lane has read its scores: the words may be reused
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) {
            float* zq = sp<float>(zs_off + qi * ZQ * 4);
            unsigned short* zh = reinterpret_cast<unsigned short*>(zq);
            if (n_spans > 1 && lane == 0 && qi < nq) { d.part[qi] = m[qi]; d.part[NQ + qi] = sum[qi]; }     // for the combine
            const float inv = (n_spans == 1) ? 1.0f / sum[qi] : 1.0f;
            const float w0 = z0[qi] * inv, w1 = z1[qi] * inv;
            if (d.S && qi < nq) {
                float* Srow = d.S + qi * S_qstride;
                if (in0) Srow[lane] = w0;
                if (two && in1) Srow[lane + 32] = w1;
            }
            if (PACK) {
                if (lane < n_pad) {
                    const __nv_bfloat16 hi = __float2bfloat16_rn(w0);
                    const __nv_bfloat16 lo = __float2bfloat16_rn(w0 - __bfloat162float(hi));
                    const int at = packed_slot(lane);
                    zh[at] = *reinterpret_cast<const unsigned short*>(&hi);
                    zh[at + 4] = *reinterpret_cast<const unsigned short*>(&lo);
                }
                if (two && lane + 32 < n_pad) {
                    const __nv_bfloat16 hi = __float2bfloat16_rn(w1);
                    const __nv_bfloat16 lo = __float2bfloat16_rn(w1 - __bfloat162float(hi));
                    const int at = packed_slot(lane + 32);
                    zh[at] = *reinterpret_cast<const unsigned short*>(&hi);
                    zh[at + 4] = *reinterpret_cast<const unsigned short*>(&lo);
                }
            } else {
                if (lane < n_pad) zq[lane] = w0;
                if (two && lane + 32 < n_pad) zq[lane + 32] = w1;
            }
        }
        __syncwarp();
        return;
    }
#pragma unroll 1
    for (int qi = 0; qi < nq; ++qi) {        // long spans: row by row; rows of absent queries are never stored
        float* zq = sp<float>(zs_off + qi * ZQ * 4);
        unsigned short* zh = reinterpret_cast<unsigned short*>(zq);
        float* Srow = d.S ? d.S + qi * S_qstride : nullptr;
        float m = -INFINITY;
#pragma unroll 1
        for (int jj = lane; jj < n; jj += 32) m = fmaxf(m, zq[jj]);
        m = warp_max(m);
        float s = 0.f;
#pragma unroll 1
        for (int jj = lane; jj < n; jj += 32) { const float e = exp2f(zq[jj] - m); zq[jj] = e; s += e; }
        s = warp_sum(s);
        if (n_spans > 1 && lane == 0) { d.part[qi] = m; d.part[NQ + qi] = s; }
        const float inv = (n_spans == 1) ? 1.0f / s : 1.0f;
#pragma unroll 1
        for (int j0 = 0; j0 < n_pad; j0 += 32) {      // warp-uniform trip count
            const int jj = j0 + lane;
            const float w = jj < n ? zq[jj] * inv : 0.f;
            if (Srow && jj < n) Srow[jj] = w;
            if (PACK) {
                __syncwarp();
                if (jj < n_pad) {
                    const __nv_bfloat16 hi = __float2bfloat16_rn(w);
                    const __nv_bfloat16 lo = __float2bfloat16_rn(w - __bfloat162float(hi));
                    const int at = packed_slot(jj);
                    zh[at] = *reinterpret_cast<const unsigned short*>(&hi);
                    zh[at + 4] = *reinterpret_cast<const unsigned short*>(&lo);
                }
            } else if (jj < n_pad) {
                zq[jj] = w;
            }
        }
    }
    __syncwarp();
}

// float32 items: packed two-wide FMAs on the CUDA cores (rows in natural chunk order).
template <typename T>
template <int NQ>
__device__ bool FusedWarp<T>::process(const ItemDesc& d) {
    constexpr int ZQ = kZFloats / NQ;          // score slots per query row
    constexpr int HDR = (2 * NQ + 3) / 4 * 4;  // (max, sum) per query ahead of a span's partial sums
    const KindParams& kp = p.k[d.kind];
    const int n = d.n, nq = d.nq, has_new = d.has_new, pi = d.pi;
    const int g = lane / LPR, c = lane % LPR;   // row of a block this lane reads, and its 16-byte chunk
    float* zs = sp<float>(zs_off);

    // ---- key tiles: scores into zs.  The first tile also carries the query rows.
    float2 q2[NQ][NP];
    for (int s0 = 0; s0 < n;) {
        const uint32_t st_o = acquire();
        if (st_o == kNoTile) return false;
        const char* st = sp<char>(st_o);
        const int r = min(s0 == 0 ? QROW : TR, n - s0);
        if (s0 == 0) {
            const float sc = p.scale_log2e;
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) {
                if (qi < nq) {
                    P::load(*reinterpret_cast<const uint4*>(st + (QROW + qi) * ROW_BYTES + c * 16), q2[qi]);
#pragma unroll
                    for (int e = 0; e < NP; ++e) { q2[qi][e].x *= sc; q2[qi][e].y *= sc; }
                } else {
#pragma unroll
                    for (int e = 0; e < NP; ++e) q2[qi][e] = make_float2(0.f, 0.f);
                }
            }
        }
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
                if (with_new && d.lead && j == r - 1)
                    *reinterpret_cast<uint4*>(const_cast<char*>(d.srcK) + (n - 1) * ROW_BYTES + c * 16) = kv[u];
            }
        }
        s0 += r;
        release();
    }
    __syncwarp();

    const int n_spans = d.n_spans;
    softmax_span<NQ, false>(d, n, n);

    // ---- value tiles, layer by layer (score rows of absent queries hold zeros)
    const long long O_qstride = (long long)p.H * ROW_BYTES;
    for (int l = 0; l < pi; ++l) {
        float2 acc[NQ][NP];
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi)
#pragma unroll
            for (int e = 0; e < NP; ++e) acc[qi][e] = make_float2(0.f, 0.f);
        for (int s0 = 0; s0 < n; s0 += TR) {
            const uint32_t st_o = acquire();
            if (st_o == kNoTile) return false;
            const char* st = sp<char>(st_o);
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
                            *reinterpret_cast<uint4*>(const_cast<char*>(d.srcV) + (long long)l * kp.plane_bytes +
                                                      (n - 1) * ROW_BYTES + c * 16) = vv[u];
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
                        *reinterpret_cast<uint4*>(d.O + l * kp.layer_bytes + qi * O_qstride + c * 16) = P::store(acc[qi]);
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
    __threadfence();
    __syncwarp();
    int t = 0;
    if (lane == 0) t = atomicAdd(p.tickets + d.row_id, 1);
    t = __shfl_sync(0xffffffffu, t, 0);
    if (t == n_spans - 1) combine_spans<T, NQ>(p, d, zs_off, lane);
    return true;
}

// bf16 items on the tensor cores (mma.sync m16n8k16, float32 accumulate).  Neither product
// is a dense GEMM: the tensor cores are used because one 16-row block of a tile then costs
// a handful of instructions (4 ldmatrix + 4 mma for the scores, 4 ldmatrix + 16 mma for one
// layer's S.V) instead of a hundred or more unpack/FMA/shuffle instructions, and the step
// is bound by instruction issue, not by tensor throughput.
//   scores:  D[16 positions x 8 queries] = K_tile[16 x 64] . q^T              (queries padded to 8)
//   apply:   D[16 dims x 8 queries]     += V_tile^T[16 x 16 positions] . S^T   (four dim tiles)
// S is used as a bf16 high part plus a bf16 remainder (two MMAs), packed once per item by
// the softmax, so that the weights keep about 16 bits; products and sums are float32.
// Columns of D that belong to padding queries are computed from whatever the padding lanes
// load and are never stored.
template <typename T>
template <int NQ>
__device__ bool FusedWarp<T>::process_mma(const ItemDesc& d) {
    static_assert(sizeof(T) == 2, "tensor-core path is for bf16 rows");
    constexpr int ZQ = kZFloats / NQ;
    constexpr int HDR = (2 * NQ + 3) / 4 * 4;
    const int n = d.n, nq = d.nq, has_new = d.has_new, pi = d.pi;
    const int tig = lane & 3, gid = lane >> 2;                 // mma fragment coordinates
    // ldmatrix: this lane addresses row lrow of a 16-row block and, for the pair of 16-byte
    // chunks 2x, 2x+1, the chunk 2x + (lane >> 4).  Cached rows keep chunk c at c ^ (row & 7)
    // (row & 7 == lane & 7 here); this step's own row arrives in natural order, so a lane that
    // addresses it takes the permutation out again (new_fix).
    const int lrow = (lane & 7) + ((lane >> 3) & 1) * 8;
    const uint32_t new_fix = (uint32_t)(lane & 7) << 4;
    uint32_t ld_off[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) ld_off[x] = (uint32_t)(lrow * 128 + (((2 * x + (lane >> 4)) ^ (lane & 7)) << 4));

    // ---- key tiles: scores into zs (log2 domain).  The first tile also carries the query rows
    // (natural chunk order), read as B fragments (k = dims, n = query).
    uint32_t qb[4][2];
    const float sc = p.scale_log2e;
    const uint32_t zk = zs_off + ((2 * tig) * ZQ + gid) * 4;   // this lane's score slots: queries 2tig, 2tig+1; positions gid, gid+8
    for (int s0 = 0; s0 < n;) {
        const uint32_t st = acquire();
        if (st == kNoTile) return false;
        const int r = min(s0 == 0 ? QROW : TR, n - s0);
        if (s0 == 0) {
            const uint32_t qrow = st + (QROW + (gid < nq ? gid : 0)) * 128 + 4 * tig;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                qb[ks][0] = *sp<uint32_t>(qrow + 32 * ks);
                qb[ks][1] = *sp<uint32_t>(qrow + 32 * ks + 16);
            }
        }
        const int new_row = (has_new && s0 + r == n) ? r - 1 : -1;     // where this step's key row sits in the tile
        if (new_row >= 0 && d.lead && lane < 8)                        // into the cache, chunk-permuted
            *reinterpret_cast<uint4*>(const_cast<char*>(d.srcK) + (n - 1) * 128 + ((lane ^ (new_row & 7)) << 4)) =
                *sp<uint4>(st + new_row * 128 + lane * 16);
        const uint32_t st_s = sm_base + st;
#pragma unroll 1
        for (int b0 = 0; b0 < r; b0 += 16) {
            const uint32_t fix = (b0 + lrow == new_row) ? new_fix : 0u;
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            uint32_t a[4][4];          // all four loads first: their latencies overlap
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) ldsm_x4(st_s + b0 * 128 + (ld_off[ks] ^ fix), a[ks]);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) mma_bf16(acc, a[ks][0], a[ks][1], a[ks][2], a[ks][3], qb[ks][0], qb[ks][1]);
            // acc[0], acc[1]: position b0+gid, queries 2tig, 2tig+1; acc[2], acc[3]: position b0+gid+8.
            // Rows of the block at or beyond r (the query rows of a first tile, stale bytes) give
            // scores that the next tile overwrites; nothing is stored beyond the span.
            const int pos = s0 + b0 + gid;
            float* z = sp<float>(zk + (s0 + b0) * 4);
            if (2 * tig < NQ) {
                if (pos < n) z[0] = acc[0] * sc;
                if (pos + 8 < n) z[8] = acc[2] * sc;
            }
            if (2 * tig + 1 < NQ) {
                if (pos < n) z[ZQ] = acc[1] * sc;
                if (pos + 8 < n) z[ZQ + 8] = acc[3] * sc;
            }
        }
        s0 += r;
        release();
    }
    __syncwarp();

    const int n_spans = d.n_spans;
    softmax_span<NQ, true>(d, n, (n + 15) & ~15);

    // ---- value tiles, layer by layer
    // B fragments: the weights of query gid at positions b0 + {2tig, 2tig+1} and b0 + {2tig+8, 2tig+9},
    // high parts and remainders, one 16-byte load per block straight from the packed words.
    // A fragments: the tile transposed by ldmatrix; this lane addresses position vrow of a block
    // and, for the dim tile x, the 16-byte chunk 2x + ((lane >> 3) & 1).
    const uint32_t za = zs_off + (gid < NQ ? gid : 0) * ZQ * 4 + tig * 16;
    const int vrow = (lane & 7) + ((lane >> 4) << 3);
    uint32_t vd_off[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) vd_off[x] = (uint32_t)(vrow * 128 + (((2 * x + ((lane >> 3) & 1)) ^ (lane & 7)) << 4));
    const KindParams& kp = p.k[d.kind];
    const long long plane_bytes = kp.plane_bytes, layer_bytes = kp.layer_bytes;
    char* vlast = const_cast<char*>(d.srcV) + (n - 1) * 128;      // where this step's value row goes
    // output: this lane ends up with a pair of adjacent dims of one query (see below)
    const int odd = gid & 1;
    const int q_mine = NQ == 1 ? 0 : 2 * tig + odd;
    const bool q_store = NQ == 1 ? (tig == 0 && !odd) : (q_mine < nq);
    char* op = d.O + q_mine * ((long long)p.H * 128) + (gid - odd) * 2;
#pragma unroll 1
    for (int l = 0; l < pi; ++l) {
        float acc[4][4];
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[x][e] = 0.f;
#pragma unroll 1
        for (int s0 = 0; s0 < n; s0 += TR) {
            const uint32_t st = acquire();
            if (st == kNoTile) return false;
            const int r = min(TR, n - s0);
            const int new_row = (has_new && s0 + r == n) ? r - 1 : -1;
            if (new_row >= 0 && lane < 8)
                *reinterpret_cast<uint4*>(vlast + ((lane ^ (new_row & 7)) << 4)) = *sp<uint4>(st + new_row * 128 + lane * 16);
            const uint32_t st_s = sm_base + st;
#pragma unroll 1
            for (int b0 = 0; b0 < r; b0 += 16) {
                const uint4 w = *sp<uint4>(za + (s0 + b0) * 4);      // (high b0, high b1, remainder b0, remainder b1)
                // rows at or beyond r hold stale bytes: their weights are zero, but 0 x NaN would not be,
                // so those lanes address a row of zeros instead
                const int row = b0 + vrow;
                const uint32_t fix = (row == new_row) ? new_fix : 0u;
                const uint32_t blk = st_s + b0 * 128;
                uint32_t a[4][4];      // all four loads first: their latencies overlap
#pragma unroll
                for (int x = 0; x < 4; ++x) ldsm_x4_t(row < r ? blk + (vd_off[x] ^ fix) : zero_row, a[x]);
#pragma unroll
                for (int x = 0; x < 4; ++x) mma_bf16(acc[x], a[x][0], a[x][1], a[x][2], a[x][3], w.x, w.y);
#pragma unroll
                for (int x = 0; x < 4; ++x) mma_bf16(acc[x], a[x][0], a[x][1], a[x][2], a[x][3], w.z, w.w);
            }
            release();
        }
        // acc[x][0], [1]: dim 16x + gid of queries 2tig, 2tig+1; acc[x][2], [3]: dim 16x + gid + 8
        if (n_spans == 1) {
            // lanes gid and gid ^ 1 hold adjacent dims: the even one collects the pair of query 2tig,
            // the odd one the pair of query 2tig + 1 (one query: only the even lanes of tig 0 store)
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t packed;
                    if (NQ == 1) {
                        const float up = __shfl_down_sync(0xffffffffu, acc[x][2 * h], 4);
                        packed = pack_bf16x2(acc[x][2 * h], up);
                    } else {
                        const float got = __shfl_xor_sync(0xffffffffu, odd ? acc[x][2 * h] : acc[x][2 * h + 1], 4);
                        packed = odd ? pack_bf16x2(got, acc[x][2 * h + 1]) : pack_bf16x2(acc[x][2 * h], got);
                    }
                    if (q_store) *reinterpret_cast<uint32_t*>(op + (16 * x + 8 * h) * 2) = packed;
                }
        } else {
            float* pp = d.part + HDR + ((long long)l * NQ + 2 * tig) * kDh + gid;
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    if (2 * tig < nq) pp[16 * x + 8 * h] = acc[x][2 * h];
                    if (2 * tig + 1 < nq) pp[kDh + 16 * x + 8 * h] = acc[x][2 * h + 1];
                }
        }
        vlast += plane_bytes;
        op += layer_bytes;
    }
    if (n_spans == 1) return true;

    __threadfence();
    __syncwarp();
    int t = 0;
    if (lane == 0) t = atomicAdd(p.tickets + d.row_id, 1);
    t = __shfl_sync(0xffffffffu, t, 0);
    if (t == n_spans - 1) combine_spans<T, NQ>(p, d, zs_off, lane);
    return true;
}

// The last span of a split row: softmax weights across spans, then S and every layer's O.
// Rare (split rows only) and long: kept out of line so that the hot loops stay small.
template <typename T, int NQ>
__device__ __noinline__ void combine_spans(const StepParams& p, const ItemDesc& d, uint32_t zs_off, int lane) {
    constexpr int HDR = (2 * NQ + 3) / 4 * 4;
    constexpr int ROW_BYTES = FusedGeom<T>::ROW_BYTES;
    __threadfence();
    const KindParams& kp = p.k[d.kind];
    const int n_spans = d.n_spans, nq = d.nq, stride = (int)kp.part_stride;
    const float* row_part = d.part - (long long)d.span * stride;
    const int span_len = (int)kp.span;
    const long long S_qstride = (long long)p.H * kp.S_ld, O_qstride = (long long)p.H * ROW_BYTES;
    // zs[sp * NQ + qi] = exp2(m_sp - M) / total  (zs is free: every layer of this span is done)
    float* zs = sp<float>(zs_off);
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
            float* Srow = d.S - d.span * span_len + qi * S_qstride;      // d.S starts at this span's first position
#pragma unroll 1
            for (int j = lane; j < d.len; j += 32) Srow[j] = __ldcg(Srow + j) * zs[(j / span_len) * NQ + qi];
        }
    }
    // every layer's output: E = pi*NQ*64 floats per span, four per lane per pass
    const int E = d.pi * NQ * kDh;
#pragma unroll 1
    for (int e0 = lane * 4; e0 < E; e0 += 128) {
        const int qi = (e0 / kDh) % NQ;
        if (qi >= nq) continue;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        const float* src = row_part + HDR + e0;
        int sn = 0;
#pragma unroll 1
        for (; sn + 4 <= n_spans; sn += 4) {
            float4 x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) x[u] = __ldcg(reinterpret_cast<const float4*>(src + (long long)(sn + u) * stride));
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float f = zs[(sn + u) * NQ + qi];
                a.x = fmaf(f, x[u].x, a.x); a.y = fmaf(f, x[u].y, a.y); a.z = fmaf(f, x[u].z, a.z); a.w = fmaf(f, x[u].w, a.w);
            }
        }
#pragma unroll 1
        for (; sn < n_spans; ++sn) {
            const float4 x = __ldcg(reinterpret_cast<const float4*>(src + (long long)sn * stride));
            const float f = zs[sn * NQ + qi];
            a.x = fmaf(f, x.x, a.x); a.y = fmaf(f, x.y, a.y); a.z = fmaf(f, x.z, a.z); a.w = fmaf(f, x.w, a.w);
        }
        const int ly = e0 / (NQ * kDh), col = e0 % kDh;
        char* op = d.O + ly * kp.layer_bytes + qi * O_qstride + col * (int)sizeof(T);
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

// AAN running average (Table 6 pairing): element-wise.  A CTA's share is cut into chunks of
// 32 lanes x 4 columns that its warps take from a counter in shared memory once they have no
// attention item left (or never had one), so that the averages run beside the attention items'
// chains and not ahead of them.  Called by whole warps; *aan_next starts at zero.
template <typename T>
__device__ __forceinline__ void aan_chunks(const StepParams& p, int lane, unsigned* aan_next) {
    if (!p.x_aan) return;
    const int d = p.H * kDh, d4 = d >> 2;
    const long long total = (long long)p.n_aan_layers * p.n_aan_seqs * d4;
    const long long n_chunks = (total + 31) / 32;
    for (;;) {
        unsigned j = 0;
        if (lane == 0) j = atomicAdd(aan_next, 1u);
        j = __shfl_sync(0xffffffffu, j, 0);
        const long long ck = (long long)blockIdx.x + (long long)j * gridDim.x;
        if (ck >= n_chunks) break;
        const long long u = ck * 32 + lane;
        if (u >= total) continue;
        const int c4 = (int)(u % d4);
        const int item = (int)((u / d4) % p.n_aan_seqs);
        const int lr = (int)(u / ((long long)d4 * p.n_aan_seqs));
        const int id = p.aan_ids[item], t = p.t_aan[item];
        if (id < 0 || id >= p.aan_max_seqs) { if (c4 == 0 && lr == 0) record_error(p.err, TAG_AAN, item, id, p.aan_max_seqs); continue; }
        if (t < 1 || t > p.aan_max_t) { if (c4 == 0 && lr == 0) record_error(p.err, TAG_AAN, item, t, p.aan_max_t); continue; }
        const long long io = ((long long)lr * p.n_aan_seqs + item) * d + c4 * 4;
        float xv[4];
        if (sizeof(T) == 2) {
            const uint2 raw = *reinterpret_cast<const uint2*>(p.x_aan + io * 2);
            xv[0] = __uint_as_float(raw.x << 16); xv[1] = __uint_as_float(raw.x & 0xffff0000u);
            xv[2] = __uint_as_float(raw.y << 16); xv[3] = __uint_as_float(raw.y & 0xffff0000u);
        } else {
            const float4 raw = *reinterpret_cast<const float4*>(p.x_aan + io * 4);
            xv[0] = raw.x; xv[1] = raw.y; xv[2] = raw.z; xv[3] = raw.w;
        }
        float4* sum = reinterpret_cast<float4*>(p.aan_sum + ((long long)lr * p.aan_max_seqs + id) * d + c4 * 4);
        float4 s = (t == 1) ? make_float4(0.f, 0.f, 0.f, 0.f) : *sum;
        s.x += xv[0]; s.y += xv[1]; s.z += xv[2]; s.w += xv[3];
        *sum = s;
        const float ft = (float)t;
        const float o[4] = {s.x / ft, s.y / ft, s.z / ft, s.w / ft};
        if (sizeof(T) == 2) {
            __nv_bfloat162 a = __floats2bfloat162_rn(o[0], o[1]), b = __floats2bfloat162_rn(o[2], o[3]);
            uint2 r; r.x = *reinterpret_cast<uint32_t*>(&a); r.y = *reinterpret_cast<uint32_t*>(&b);
            *reinterpret_cast<uint2*>(p.aan_out + io * 2) = r;
        } else {
            *reinterpret_cast<float4*>(p.aan_out + io * 4) = make_float4(o[0], o[1], o[2], o[3]);
        }
    }
}

constexpr int kCtaItems = 144;      // decoded items a CTA holds at a time (at most 255: the warps queue them by byte)
constexpr size_t fused_smem_bytes() {
    return (size_t)kFusedWarps * (kFusedStages * kStageBytes + kZFloats * sizeof(float) + kFusedStages * sizeof(uint64_t)) +
           128 /* a row of zeros */ + (size_t)kCtaItems * sizeof(ItemDesc);
}

template <typename T, int NQE>
__global__ void __launch_bounds__(kFusedWarps * 32, 1) decode_step_kernel(const __grid_constant__ StepParams p) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    // The launch allows programmatic stream serialization: the next kernel of the stream may be
    // scheduled onto SMs as this grid leaves them, and this grid may have been scheduled while
    // its predecessor was still finishing.  Nothing is read from or written to global memory
    // until the predecessor has completed and its writes are visible (the wait below); only the
    // set-up of shared memory runs ahead of it.  Without the launch attribute both are no-ops.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // layout of san_smem: the warps' rings, their score slots, their barriers, a row of zeros, the CTA's items
    constexpr uint32_t kZsAll = kFusedWarps * kFusedStages * kStageBytes;
    constexpr uint32_t kBarsAll = kZsAll + kFusedWarps * kZFloats * (uint32_t)sizeof(float);
    constexpr uint32_t kZeroRow = kBarsAll + kFusedWarps * kFusedStages * (uint32_t)sizeof(uint64_t);
    constexpr uint32_t kDescsAll = kZeroRow + 128;
    if (threadIdx.x < 32) *sp<uint32_t>(kZeroRow + threadIdx.x * 4) = 0u;      // read after the first CTA barrier
    if (lane == 0) {
        for (int s = 0; s < kFusedStages; ++s) mbar_init(sp<uint64_t>(kBarsAll + ((uint32_t)warp * kFusedStages + s) * 8), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // ---- AAN running average: see aan_chunks
    __shared__ unsigned aan_next;
    if (threadIdx.x == 0) aan_next = 0u;
    auto aan_part = [&]() { aan_chunks<T>(p, lane, &aan_next); };
    if (p.n_items == 0) { __syncthreads(); aan_part(); return; }

    // ---- attention items.  CTA b owns list slots b, b + G, b + 2G, ...  It takes them in rounds
    // of kCtaItems slots: every thread decodes one slot, the survivors are packed in list order
    // (big items first), then the warps drain them through a shared counter.
    __shared__ unsigned q_next, warp_count[kFusedWarps];
    ItemDesc* descs = sp<ItemDesc>(kDescsAll);

    FusedWarp<T> w(p);
    w.sm_base = smem_u32(san_smem);
    w.ring = (uint32_t)warp * kFusedStages * kStageBytes;
    w.bars = kBarsAll + (uint32_t)warp * kFusedStages * 8;
    w.zs_off = kZsAll + (uint32_t)warp * kZFloats * 4;
    w.descs_off = kDescsAll; w.q_next = &q_next; w.zero_row = w.sm_base + kZeroRow;
    w.lane = lane;
    w.p_stage = 0; w.c_stage = 0; w.c_par = 0; w.dead = false; w.p_active = false;

    const unsigned long long my_slots = (p.n_items > blockIdx.x) ? ((unsigned long long)p.n_items - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    if (my_slots == 0) { __syncthreads(); aan_part(); }     // a CTA without attention items still has its share of the averages
    for (unsigned long long k0 = 0; k0 < my_slots; k0 += kCtaItems) {
        // -- decode: thread t takes slot k0 + t; survivors keep their order
        ItemDesc mine;
        bool ok = false;
        if (threadIdx.x < kCtaItems && k0 + threadIdx.x < my_slots)
            ok = decode_item<FusedGeom<T>::ROW_BYTES>(p, (unsigned)((k0 + threadIdx.x) * gridDim.x + blockIdx.x), &mine);
        const unsigned ballot = __ballot_sync(0xffffffffu, ok);
        if (lane == 0) warp_count[warp] = __popc(ballot);
        __syncthreads();                                 // also: every warp is done with the previous round's items
        if (threadIdx.x == 0) q_next = kFusedWarps;      // the first kFusedWarps items go to the warps directly
        // lane i holds warp i's count: survivors ahead of this warp's, and all of them
        static_assert(kFusedWarps <= 32, "one lane per warp");
        const unsigned cnt = lane < kFusedWarps ? warp_count[lane] : 0u;
        unsigned before = lane < warp ? cnt : 0u, total = cnt;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            before += __shfl_xor_sync(0xffffffffu, before, o);
            total += __shfl_xor_sync(0xffffffffu, total, o);
        }
        if (ok) descs[before + __popc(ballot & ((1u << lane) - 1u))] = mine;
        __syncthreads();
        // -- drain
        w.n_valid = w.dead ? 0u : total;
        w.nx_idx = (unsigned)warp;
        w.fifo = 0ull; w.fifo_n = 0;
        w.next_item();
#pragma unroll 1
        for (int s = 0; s < kFusedStages; ++s) w.produce();
        while (w.fifo_n > 0 && !w.dead) {
            const ItemDesc& d = w.desc((unsigned)(w.fifo & 0xffull));
            w.fifo >>= 8; w.fifo_n -= 1;
            if constexpr (sizeof(T) == 2) {
                if (NQE > 1 && d.kind) w.template process_mma<NQE>(d); else w.template process_mma<1>(d);
            } else {
                if (NQE > 1 && d.kind) w.template process<NQE>(d); else w.template process<1>(d);
            }
        }
        if (k0 == 0) aan_part();      // warps that are out of attention items (or never had one) take the averages
        // a warp whose wait ran out stops working but keeps meeting the CTA at the barriers above
    }
}

}  // namespace san
