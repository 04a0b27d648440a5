// One decode step in one launch, bf16, for rows of any length: cache append, weights (Eq. 1)
// and apply (Eq. 2 with Eq. 4) for every block of both attention kinds, plus the AAN running
// average (Table 6 pairing).
//
// Work is a flat list of UNITS: [AAN chunks][encoder-memory units][self-attention units].  An
// attention unit is one span of one (block, id, head, layer group) row; short rows are one
// span, long rows are cut into 2 or 4 spans handled by neighbouring warps.  A CTA is four
// TEAMS, each one producer warp feeding four consumer warps through its own ring in shared
// memory.  A producer takes BUNDLES of up to four consecutive units from a counter in global
// memory (whole bundles while plenty of work is left, smaller ones towards the end so that the
// SMs finish together), decodes them one unit per lane, and streams their cache rows into the
// ring with bulk asynchronous copies: one SLOT per (plane, tile of positions) holds that tile
// of all four units, is filled by one copy instruction (one lane per unit) and completes on one
// mbarrier.  Issuing a bulk copy holds a warp for several hundred cycles whatever its size,
// which is why the copies are issued by warps that do nothing else and why a slot is one
// instruction.  Each consumer warp owns one unit of the bundle: it fetches the unit's query
// rows and this step's new key/value rows itself (16-byte asynchronous copies into a scratch
// row set of its own), waits for the slot, scores its rows (tensor cores, mma.sync m16n8k16,
// float32 accumulate), releases the slot, runs the softmax, then applies the weights to the
// value tiles of every layer of the unit as their slots arrive.  The spans of a long row
// exchange (max, sum) and their partial outputs through shared memory inside the team;
// nothing goes through global memory.
//
// Every wait (full / empty slot barriers, the team's exchange barrier) is bounded: a wait
// that runs out records SAN_ERR_TIMEOUT, raises a CTA-wide flag that makes every other wait
// give up at once, and the producers leave after their copies in flight have landed.
#pragma once

#include "san_fused.cuh"

namespace san {

constexpr int kTeams = 4;
constexpr int kTeamWarps = 2;                                  // consumer warps of a team = units per bundle
constexpr int kUnitRows = 4;                                   // a unit is up to four rows (heads) of one (block, id)
constexpr int kStepConsumers = kTeams * kTeamWarps;
constexpr int kStepWarps = kStepConsumers + kTeams;            // + one producer per team
constexpr int kNS = 8;                                         // slots (and bundles) a team may have outstanding
constexpr int kRingPad = 2048;                                 // a 16-row ldmatrix block may read past a unit's last row
constexpr int kAanChunk = 256;                                 // elements of one AAN unit (8 per lane)
// Apply S as a bf16 high part plus a bf16 remainder (two MMAs per tile) or as the high part alone.
// Outputs are bf16: their own rounding (2^-9 relative) is what the comparison with the float64
// reference shows either way (3.9e-3 normwise at worst on all workloads, tolerance 1e-2), so the
// remainder is left out.
constexpr bool kWeightRemainder = false;
constexpr int kXq = 16;                                        // query rows the exchange area has room for per unit

enum { TAG_TEAM = 8 };
enum { UK_SELF = 0, UK_ENC = 1, UK_AAN = 2, UK_IDLE = 3 };

struct TeamKind {
    const char* q; const char* K; const char* V;      // queries; key / value plane 0 of the kind
    const char* knew; const char* vnew;               // this step's rows (self only, else null)
    float* S; char* O;                                 // S may be null
    const int* ids; const int* lens;                   // lens: source lengths (enc-dec) or write positions (self)
    long long plane_bytes;                             // between cache planes
    long long layer_bytes;                             // between layers in O and v_new / blocks in k_new
    long long S_ld;                                    // floats between S rows
    unsigned panel_bytes;                              // capacity * 128: one (id, head) panel
    unsigned n_it, nq, len_bias, max_ids, bound;
    unsigned q_first, q_stride_items;                  // first query row this launch covers; queries per item in q/S/O
    unsigned spr_log2;                                 // spans per row = 1 << spr_log2 (at most kTeamWarps)
    unsigned lg_size, v_by_block;
    unsigned rpu;                                      // rows (consecutive heads of one id) per unit: 1, 2 or 4; 1 when rows are split into spans
    unsigned n_rowlg;                                  // (block, row group, layer group) triples
    unsigned tile_pos;                                 // positions per tile (multiple of 16)
    unsigned zq;                                       // floats between the score rows of two queries
    unsigned n_units;                                  // padded to a multiple of kTeamWarps
    FastDiv div_lg, div_rows, div_h;
    unsigned char first[SAN_MAX_LAYERS], size[SAN_MAX_LAYERS];
};

struct TeamParams {
    TeamKind k[2];                                     // [0] self, [1] enc-dec
    unsigned n_aan_units, n_enc_units, n_units;        // list order: AAN, enc-dec, self
    int H;
    int* err; int* queue;                              // queue[0]: next unit; queue[1]: producers done
    float scale_log2e;
    unsigned grab_teams;                               // bundles shrink once fewer than grab_teams * kTeamWarps units are left
    // shared-memory layout (byte offsets); every team has its own ring
    unsigned ring_bytes, ring_stride, off_zs, zs_bytes, off_scr, scr_bytes, off_xo, xo_unit_floats, off_desc, off_bars, off_zero;
    // AAN (absent when x_aan == null)
    const char* x_aan; const int* t_aan; const int* aan_ids; float* aan_sum; char* aan_out;
    int n_aan_layers, n_aan_seqs, aan_max_seqs, aan_max_t, aan_chunks_per_row;
    FastDiv div_aan_chunks, div_aan_seqs;
};

// What a consumer needs to know about its unit; written by the producer lane that decoded it.
struct __align__(16) UnitDesc {
    char* dstK;               // where this step's key row goes in the cache (null: not this unit's to store)
    char* dstV;               // where this step's value row of the unit's first layer goes (null: none)
    float* S;                 // S of query 0 at the span's first position (null: not stored)
    char* O;                  // output row of (first layer, query 0)
    const char* q;            // query row 0 of the unit (further queries H * 128 bytes apart)
    const char* knew;         // this step's key row (valid when new_row >= 0)
    const char* vnew;         // this step's value row of the unit's first layer
    int n;                    // positions in the span
    int new_row;              // index in the span of this step's row (not yet cached), or -1
    unsigned char kind, nq, pi, tp, span, spr_log2, rows, pad1;
    unsigned int aux;         // AAN: target position t
    unsigned int pad[5];
};
static_assert(sizeof(UnitDesc) == 96, "UnitDesc is addressed as 96 bytes");

struct __align__(16) BundleHdr { int tiles, layers, sync, end; };
struct __align__(16) SlotDesc { uint32_t base; uint16_t off[kTeamWarps]; uint32_t pad; };
static_assert(sizeof(SlotDesc) == 16, "SlotDesc is addressed as 16 bytes");

constexpr uint32_t kUnitDescBytes = (uint32_t)sizeof(UnitDesc);
constexpr uint32_t kTeamDescBytes = kNS * (kTeamWarps * kUnitDescBytes + (uint32_t)sizeof(BundleHdr) + (uint32_t)sizeof(SlotDesc));
// barriers: per team full[kNS], empty[kNS], ready[kNS] (a bundle's descriptors are written), exchange[1];
// then the CTA's dead flag
constexpr uint32_t kTeamBarBytes = (3 * kNS + 1) * 8;
// exchange area of a team: two output buffers of kTeamWarps units, then (max, sum) per unit and query
__host__ __device__ constexpr uint32_t team_xch_bytes(uint32_t xo_unit_floats) {
    return 2u * kTeamWarps * xo_unit_floats * 4u + kTeamWarps * kXq * 2u * 4u;
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

// ------------------------------------------------------------------------------ shared views
struct StepSmem {
    uint32_t sm_base;         // shared-space address of san_smem
    uint32_t off_desc, off_bars;
    __device__ __forceinline__ uint32_t unit_desc(int team, int bslot, int u) const {
        return off_desc + (uint32_t)team * kTeamDescBytes + (uint32_t)(bslot * kTeamWarps + u) * kUnitDescBytes;
    }
    __device__ __forceinline__ uint32_t bundle_hdr(int team, int bslot) const {
        return off_desc + (uint32_t)team * kTeamDescBytes + kNS * kTeamWarps * kUnitDescBytes + (uint32_t)bslot * 16u;
    }
    __device__ __forceinline__ uint32_t slot_desc(int team, int slot) const {
        return off_desc + (uint32_t)team * kTeamDescBytes + kNS * (kTeamWarps * kUnitDescBytes + 16u) + (uint32_t)slot * 16u;
    }
    __device__ __forceinline__ uint32_t bar_full(int team, int slot) const { return sm_base + off_bars + (uint32_t)team * kTeamBarBytes + (uint32_t)slot * 8u; }
    __device__ __forceinline__ uint32_t bar_empty(int team, int slot) const { return sm_base + off_bars + (uint32_t)team * kTeamBarBytes + (uint32_t)(kNS + slot) * 8u; }
    __device__ __forceinline__ uint32_t bar_ready(int team, int bslot) const { return sm_base + off_bars + (uint32_t)team * kTeamBarBytes + (uint32_t)(2 * kNS + bslot) * 8u; }
    __device__ __forceinline__ uint32_t bar_xch(int team) const { return sm_base + off_bars + (uint32_t)team * kTeamBarBytes + 3u * kNS * 8u; }
    __device__ __forceinline__ volatile int* dead_flag() const { return sp<volatile int>(off_bars + kTeams * kTeamBarBytes); }
};

// try_wait that lets the hardware keep the thread suspended for a while (it returns as soon as
// the phase completes), so that a waiting warp does not use issue slots.  Measured on B200: a
// hint of 1,000,000 suspends for about 1000 cycles; without a hint the instruction returns at once.
constexpr uint32_t kWaitHint = 4000000u;
__device__ __forceinline__ bool mbar_try_wait_for(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(ns) : "memory");
    return ok != 0;
}

// Bounded wait that also gives up as soon as another warp of the CTA has given up.
__device__ __noinline__ bool step_wait_slow(uint32_t bar, uint32_t parity, volatile int* dead) {
    const long long t0 = clock64();
    do {
        if (mbar_poll(bar, parity, kWaitHint, 1024u)) return true;
        if (*dead) return false;
    } while (clock64() - t0 < 2000000000LL);
    return false;
}

// ------------------------------------------------------------------------------ the producer
// One per team.  Its ring is private, so slots retire in the order they were issued.
struct StepProducer {
    const TeamParams& p;
    StepSmem sm;
    int lane, team;
    uint32_t ring0;                           // offset of the team's ring in san_smem
    uint32_t head_v, tail_v, head_p;          // virtual byte counters and the physical write offset (same in every lane)
    uint32_t n_slots, n_retired, n_bundles;   // slots issued / retired, bundles issued
    uint32_t rec_end_v;                       // lane i: head_v after the slot with sequence number i (mod kNS)
    bool dead;

    __device__ StepProducer(const TeamParams& pp) : p(pp) {}

    __device__ __forceinline__ void fail(int where) {
        if (lane == 0 && atomicCAS(&p.err[0], 0, (int)SAN_ERR_TIMEOUT) == 0) { p.err[1] = TAG_TEAM; p.err[2] = where; }
        *sm.dead_flag() = 1;
        dead = true;
    }
    // The oldest outstanding slot has been read by all its consumers: its bytes and its index are free.
    __device__ __forceinline__ void retire_oldest() {
        const uint32_t seq = n_retired;
        const uint32_t end_v = __shfl_sync(0xffffffffu, rec_end_v, seq % kNS);
        const uint32_t bar = sm.bar_empty(team, (int)(seq % kNS));
        const uint32_t par = (seq / kNS) & 1u;
        if (!mbar_try_wait(bar, par) && !step_wait_slow(bar, par, sm.dead_flag())) { fail(1); return; }
        tail_v = end_v;
        n_retired += 1;
    }
    // Slot index n_slots % kNS is free again once the slot kNS before it has been retired.
    __device__ __forceinline__ void ensure_slot() {
        while (!dead && n_retired + kNS <= n_slots) retire_oldest();
    }
    // `bytes` contiguous bytes of the ring; returns the offset in san_smem.
    __device__ __forceinline__ uint32_t alloc(uint32_t bytes) {
        if (head_p + bytes > p.ring_bytes) { head_v += p.ring_bytes - head_p; head_p = 0; }
        while (!dead && n_retired < n_slots && head_v + bytes - tail_v > p.ring_bytes) retire_oldest();
        if (n_retired == n_slots) tail_v = head_v;       // nothing outstanding: the whole ring is free
        const uint32_t at = ring0 + head_p;
        head_v += bytes; head_p += bytes;
        return at;
    }
    __device__ __forceinline__ void issued() {
        if ((uint32_t)lane == n_slots % kNS) rec_end_v = head_v;
        n_slots += 1;
    }
};

// What the producer lane of a unit keeps about it.
struct ProdUnit {
    const char* srcK; const char* srcV;
    long long plane_bytes;
    unsigned panel_bytes;
    int n, pi, tp, new_row, kind, tiles, spr_log2, rows;
};

// Where unit g sits in the work list, and the entries of the id and length arrays that it
// depends on.  Worked out (and the two entries loaded) one bundle ahead of the decode, so that
// their latency is not on the producer's path.
struct UnitIdx {
    int kind;                 // UK_SELF, UK_ENC, UK_AAN, or UK_IDLE for padding
    unsigned item, h, block, lg, span;      // AAN: item, chunk (in h), layer (in block)
    int id, len;
};

__device__ __forceinline__ void unit_index(const TeamParams& p, unsigned g, bool in_bundle, UnitIdx* ui) {
    ui->kind = UK_IDLE; ui->item = ui->h = ui->block = ui->lg = ui->span = 0; ui->id = -1; ui->len = 0;
    if (!in_bundle || g >= p.n_units) return;
    if (g < p.n_aan_units) {
        unsigned rowi, chunk, lr, item;
        p.div_aan_chunks.divmod(g, &rowi, &chunk);
        p.div_aan_seqs.divmod(rowi, &lr, &item);
        if (lr >= (unsigned)p.n_aan_layers) return;                      // padding
        ui->kind = UK_AAN; ui->item = item; ui->h = chunk; ui->block = lr;
        ui->id = p.aan_ids[item]; ui->len = p.t_aan[item];
        return;
    }
    const int enc = g < p.n_aan_units + p.n_enc_units;
    const TeamKind& kp = p.k[enc];
    const unsigned x = g - p.n_aan_units - (enc ? 0u : p.n_enc_units);
    const unsigned rowlg = x >> kp.spr_log2;
    if (rowlg >= kp.n_rowlg) return;                                     // padding
    unsigned rowb, row;
    kp.div_lg.divmod(rowlg, &rowb, &ui->lg);
    kp.div_rows.divmod(rowb, &ui->block, &row);
    kp.div_h.divmod(row * kp.rpu, &ui->item, &ui->h);           // row counts groups of rpu heads (rpu divides H)
    ui->span = x & ((1u << kp.spr_log2) - 1u);
    ui->kind = enc ? UK_ENC : UK_SELF;
    ui->id = kp.ids[ui->item]; ui->len = kp.lens[ui->item];
}

// Decode of one unit by one lane: what the producer keeps (pu) and what the consumer gets (ud).
__device__ __forceinline__ void decode_unit(const TeamParams& p, const UnitIdx& ui, bool may_report, ProdUnit* pu, UnitDesc* ud) {
    pu->kind = UK_IDLE; pu->n = 0; pu->pi = 0; pu->tp = 16; pu->new_row = -1; pu->tiles = 0; pu->spr_log2 = 0; pu->rows = 0;
    pu->srcK = pu->srcV = nullptr; pu->plane_bytes = 0; pu->panel_bytes = 0;
    ud->dstK = nullptr; ud->dstV = nullptr; ud->S = nullptr; ud->O = nullptr; ud->q = ud->knew = ud->vnew = nullptr;
    ud->n = 0; ud->new_row = -1;
    ud->kind = UK_IDLE; ud->nq = 0; ud->pi = 0; ud->tp = 16; ud->span = 0; ud->spr_log2 = 0; ud->rows = 0; ud->aux = 0;
    if (ui.kind == UK_IDLE) return;
    const int id = ui.id;
    if (ui.kind == UK_AAN) {
        // ---- one chunk of one (layer, sequence) row of the running average; len holds t
        const unsigned item = ui.item, chunk = ui.h, lr = ui.block;
        const int t = ui.len;
        const bool reporter = may_report && (chunk == 0 && lr == 0);
        if (id < 0 || id >= p.aan_max_seqs) { if (reporter) record_error(p.err, TAG_AAN, (int)item, id, p.aan_max_seqs); return; }
        if (t < 1 || t > p.aan_max_t) { if (reporter) record_error(p.err, TAG_AAN, (int)item, t, p.aan_max_t); return; }
        const int d = p.H * kDh;
        const long long io = ((long long)lr * p.n_aan_seqs + item) * d + (long long)chunk * kAanChunk;
        ud->kind = UK_AAN; pu->kind = UK_AAN;
        ud->q = p.x_aan + io * 2;
        ud->dstV = reinterpret_cast<char*>(p.aan_sum + ((long long)lr * p.aan_max_seqs + id) * d + (long long)chunk * kAanChunk);
        ud->O = p.aan_out + io * 2;
        ud->n = min(kAanChunk, d - (int)chunk * kAanChunk);
        ud->aux = (unsigned)t;
        return;
    }
    const int enc = ui.kind == UK_ENC;
    const TeamKind& kp = p.k[enc];
    const unsigned span = ui.span, lg = ui.lg, block = ui.block, item = ui.item, h = ui.h;
    const int len = ui.len + (int)kp.len_bias;
    const bool reporter = may_report && (span == 0 && lg == 0 && h == 0 && block == 0);
    if ((unsigned)id >= kp.max_ids) { if (reporter) record_error(p.err, TAG_STEP, (int)item, id, (int)kp.max_ids); return; }
    if (len < 1 || len > (int)kp.bound) { if (reporter) record_error(p.err, TAG_STEP, (int)item, len, (int)kp.bound); return; }
    const unsigned size = kp.v_by_block ? 1u : kp.size[block];
    const unsigned l0 = lg * kp.lg_size;
    if (l0 >= size) return;                                              // a smaller block has fewer layer groups
    // positions of a row are dealt to its spans in runs that are multiples of 16
    const int span_len = (((len + (1 << kp.spr_log2) - 1) >> kp.spr_log2) + 15) & ~15;
    const int j0 = (int)span * span_len;
    const int j1 = min(len, j0 + span_len);
    const int n = max(0, j1 - j0);
    const unsigned H = (unsigned)p.H;
    const unsigned first = kp.first[block] + l0;
    const unsigned vplane = (kp.v_by_block ? block : kp.first[block]) + l0;
    const unsigned qrow = ((block * kp.n_it + item) * kp.q_stride_items + kp.q_first) * H + h;   // row of query 0 in q, S
    const unsigned long long panel = (unsigned long long)((unsigned)id * H + h) * kp.panel_bytes;
    const bool has_new = (kp.knew != nullptr) && n > 0 && j1 == len;
    const char* K0 = kp.K + (unsigned long long)block * (unsigned long long)kp.plane_bytes + panel;
    const char* V0 = kp.V + (unsigned long long)vplane * (unsigned long long)kp.plane_bytes + panel;
    pu->kind = ui.kind; pu->n = n; pu->pi = (int)min(kp.lg_size, size - l0);
    pu->tp = (int)kp.tile_pos; pu->new_row = has_new ? n - 1 : -1;
    pu->tiles = (n + pu->tp - 1) / pu->tp;
    pu->spr_log2 = (int)kp.spr_log2; pu->rows = (int)kp.rpu; pu->panel_bytes = kp.panel_bytes;
    pu->srcK = K0 + (unsigned)j0 * 128u; pu->srcV = V0 + (unsigned)j0 * 128u;
    pu->plane_bytes = kp.plane_bytes;
    const unsigned long long in_row = (unsigned long long)(item * H + h) * 128u;                 // self: one query per item
    ud->q = kp.q + (unsigned long long)qrow * 128u;
    ud->knew = kp.knew ? kp.knew + (unsigned long long)block * (unsigned long long)kp.layer_bytes + in_row : nullptr;
    ud->vnew = kp.vnew ? kp.vnew + (unsigned long long)first * (unsigned long long)kp.layer_bytes + in_row : nullptr;
    ud->kind = (unsigned char)pu->kind; ud->nq = (unsigned char)kp.nq; ud->pi = (unsigned char)pu->pi; ud->tp = (unsigned char)pu->tp;
    ud->span = (unsigned char)span; ud->spr_log2 = (unsigned char)kp.spr_log2; ud->rows = (unsigned char)kp.rpu;
    ud->n = n; ud->new_row = pu->new_row;
    ud->dstK = (has_new && lg == 0) ? const_cast<char*>(K0) + (unsigned)(len - 1) * 128u : nullptr;   // the lead group stores the key row
    ud->dstV = has_new ? const_cast<char*>(V0) + (unsigned)(len - 1) * 128u : nullptr;
    ud->S = (kp.S && lg == 0) ? kp.S + (unsigned long long)qrow * (unsigned long long)kp.S_ld + j0 : nullptr;
    ud->O = kp.O + (unsigned long long)vplane * (unsigned long long)kp.layer_bytes +
            (unsigned long long)((item * kp.q_stride_items + kp.q_first) * H + h) * 128u;
}

// ------------------------------------------------------------------------------ the consumer
struct StepConsumer {
    const TeamParams& p;
    StepSmem sm;
    int lane, team, u;
    uint32_t cs;              // slots of this team consumed so far
    uint32_t xs;              // exchange barriers passed so far
    uint32_t zs_off;          // this warp's score slots
    uint32_t scr_off;         // this warp's scratch rows: queries, then this step's key row, then its value rows
    uint32_t zero_row;        // shared-space address of 128 zero bytes
    bool dead;

    __device__ StepConsumer(const TeamParams& pp) : p(pp) {}

    __device__ __forceinline__ void fail(int where) {
        if (lane == 0 && atomicCAS(&p.err[0], 0, (int)SAN_ERR_TIMEOUT) == 0) { p.err[1] = TAG_TEAM; p.err[2] = where; }
        *sm.dead_flag() = 1;
        dead = true;
    }
    // Waits for the team's next slot; returns its index, or -1 after a timeout.
    __device__ __forceinline__ int acquire() {
        const int slot = (int)(cs % kNS);
        const uint32_t bar = sm.bar_full(team, slot), par = (cs / kNS) & 1u;
        if (!mbar_try_wait(bar, par) && !step_wait_slow(bar, par, sm.dead_flag())) { fail(2); return -1; }
        return slot;
    }
    // Every lane is done with the slot.
    __device__ __forceinline__ void release() {
        __syncwarp();
        if (lane == 0) mbar_arrive(sm.bar_empty(team, (int)(cs % kNS)));
        cs += 1;
    }
    // All warps of the team meet; shared-memory writes before it are visible after it.
    __device__ __forceinline__ bool team_sync() {
        const uint32_t bar = sm.bar_xch(team), par = xs & 1u;
        __syncwarp();
        if (lane == 0) mbar_arrive(bar);
        xs += 1;
        if (!mbar_try_wait(bar, par) && !step_wait_slow(bar, par, sm.dead_flag())) { fail(3); return false; }
        return true;
    }
    // Offset in san_smem of this unit's rows in the slot.
    __device__ __forceinline__ uint32_t my_rows(int slot) const {
        const uint32_t sd = sm.slot_desc(team, slot);
        return *sp<uint32_t>(sd) + (uint32_t)(*sp<uint16_t>(sd + 4 + 2 * u)) * 128u;
    }
    __device__ __forceinline__ uint32_t xch_o(int buf) const {
        return p.off_xo + (uint32_t)team * team_xch_bytes(p.xo_unit_floats) + (uint32_t)buf * (kTeamWarps * p.xo_unit_floats * 4u);
    }
    __device__ __forceinline__ uint32_t xch_ms() const {
        return p.off_xo + (uint32_t)team * team_xch_bytes(p.xo_unit_floats) + 2u * kTeamWarps * p.xo_unit_floats * 4u;
    }

    __device__ void idle(const BundleHdr& hdr);
    __device__ void aan(const UnitDesc& d);
    template <int NQ, int R> __device__ void attend(const UnitDesc& d, const BundleHdr& hdr);
    template <int NQ, int NQI> __device__ __forceinline__ bool softmax(const UnitDesc& d, const BundleHdr& hdr, int n, int n_pad, int ZQ,
                                                                       uint32_t zs_base, float* S_base, long long S_hstride, long long S_qstride, int nq);
    template <int NQ> __device__ __forceinline__ void stage_rows(const float (&acc)[4][4], int nq, int R, int hh);
    __device__ __forceinline__ void flush_rows(char* orow, int nq, int R, long long O_qstride);
};

// A warp without a unit in this bundle (or whose unit was skipped) walks the bundle's slots and
// meets the team at its exchange points.
__device__ void StepConsumer::idle(const BundleHdr& hdr) {
    for (int t = 0; t < hdr.tiles && !dead; ++t) { if (acquire() < 0) return; release(); }
    if (hdr.sync && !team_sync()) return;
    for (int l = 0; l < hdr.layers && !dead; ++l) {
        for (int t = 0; t < hdr.tiles && !dead; ++t) { if (acquire() < 0) return; release(); }
        if (hdr.sync && !team_sync()) return;
    }
}

// Running average (Table 6 pairing): sum += x; out = sum / t, 8 elements per lane.
__device__ void StepConsumer::aan(const UnitDesc& d) {
    const int e0 = lane * 8;
    if (e0 >= d.n) return;
    const uint4 raw = *reinterpret_cast<const uint4*>(d.q + e0 * 2);
    float4* sum = reinterpret_cast<float4*>(d.dstV + e0 * 4);
    const int t = (int)d.aux;
    float4 s0 = make_float4(0.f, 0.f, 0.f, 0.f), s1 = s0;
    if (t != 1) { s0 = sum[0]; s1 = sum[1]; }
    s0.x += __uint_as_float(raw.x << 16); s0.y += __uint_as_float(raw.x & 0xffff0000u);
    s0.z += __uint_as_float(raw.y << 16); s0.w += __uint_as_float(raw.y & 0xffff0000u);
    s1.x += __uint_as_float(raw.z << 16); s1.y += __uint_as_float(raw.z & 0xffff0000u);
    s1.z += __uint_as_float(raw.w << 16); s1.w += __uint_as_float(raw.w & 0xffff0000u);
    sum[0] = s0; sum[1] = s1;
    const float ft = (float)t;
    uint4 o;
    o.x = pack_bf16x2(s0.x / ft, s0.y / ft); o.y = pack_bf16x2(s0.z / ft, s0.w / ft);
    o.z = pack_bf16x2(s1.x / ft, s1.y / ft); o.w = pack_bf16x2(s1.z / ft, s1.w / ft);
    *reinterpret_cast<uint4*>(d.O + e0 * 2) = o;
}

// Softmax of n scores (log2 domain) of NQ = heads x NQI rows side by side, in place: row r
// (head r / NQI, query r % NQI) has its scores at zs_base + r * ZQ floats and its S row at
// S_base + head * S_hstride + query * S_qstride (queries at or beyond nq are carried along and
// never stored).  The weights are left as bf16 words in the order the apply
// MMAs read them (see packed_slot), zero from n up to n_pad, and are written to S.  The spans of
// a split row first exchange their (max, sum) through the team's shared memory, so every span
// normalises by the row's total.
template <int NQ, int NQI>
__device__ __forceinline__ bool StepConsumer::softmax(const UnitDesc& d, const BundleHdr& hdr, int n, int n_pad, int ZQ,
                                                      uint32_t zs_base, float* S_base, long long S_hstride, long long S_qstride, int nq) {
    const int spr = 1 << d.spr_log2;
    float* ms = sp<float>(xch_ms());     // (max, sum) of every unit of the team and query: [unit][8][2] floats
    if (n <= 64) {
        const bool two = n > 32;
        const bool in0 = lane < n, in1 = lane + 32 < n;
        float z0[NQ], z1[NQ], m[NQ], sum[NQ];
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) {
            const float* zq = sp<float>(zs_base + qi * ZQ * 4);
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
            const float mm = (n > 0) ? m[qi] : 0.f;        // an empty span: exp2(-inf - 0) = 0
            z0[qi] = exp2f(z0[qi] - mm);
            z1[qi] = exp2f(z1[qi] - mm);
            sum[qi] = z0[qi] + z1[qi];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) sum[qi] += __shfl_xor_sync(0xffffffffu, sum[qi], o);
        float inv[NQ];
        if (hdr.sync) {
            if (lane == 0) {
#pragma unroll
                for (int qi = 0; qi < NQ; ++qi) { ms[(u * kXq + qi) * 2] = m[qi]; ms[(u * kXq + qi) * 2 + 1] = sum[qi]; }
            }
            if (!team_sync()) return false;
            const int u0 = u - d.span;
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) {
                float M = -INFINITY;
                for (int s = 0; s < spr; ++s) M = fmaxf(M, ms[((u0 + s) * kXq + qi) * 2]);
                float tot = 0.f;
                for (int s = 0; s < spr; ++s) tot += ms[((u0 + s) * kXq + qi) * 2 + 1] * exp2f(ms[((u0 + s) * kXq + qi) * 2] - M);
                inv[qi] = (n > 0) ? exp2f(m[qi] - M) / tot : 0.f;
            }
        } else {
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) inv[qi] = 1.0f / sum[qi];
        }
        __syncwarp();                                   // every lane has read its scores: the words may be reused
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) {
            float* zq = sp<float>(zs_base + qi * ZQ * 4);
            unsigned short* zh = reinterpret_cast<unsigned short*>(zq);
            const float w0 = z0[qi] * inv[qi], w1 = z1[qi] * inv[qi];
            if (S_base && (qi % NQI) < nq) {
                float* Srow = S_base + (qi / NQI) * S_hstride + (qi % NQI) * S_qstride;
                if (in0) Srow[lane] = w0;
                if (two && in1) Srow[lane + 32] = w1;
            }
            if (lane < n_pad) {
                const __nv_bfloat16 hi = __float2bfloat16_rn(w0);
                const __nv_bfloat16 lo = __float2bfloat16_rn(w0 - __bfloat162float(hi));
                const int at = packed_slot(lane);
                zh[at] = *reinterpret_cast<const unsigned short*>(&hi);
                if (kWeightRemainder) zh[at + 4] = *reinterpret_cast<const unsigned short*>(&lo);
            }
            if (two && lane + 32 < n_pad) {
                const __nv_bfloat16 hi = __float2bfloat16_rn(w1);
                const __nv_bfloat16 lo = __float2bfloat16_rn(w1 - __bfloat162float(hi));
                const int at = packed_slot(lane + 32);
                zh[at] = *reinterpret_cast<const unsigned short*>(&hi);
                if (kWeightRemainder) zh[at + 4] = *reinterpret_cast<const unsigned short*>(&lo);
            }
        }
        __syncwarp();
        return true;
    }
    // long spans: row by row
    float mq[NQ], sq[NQ];
#pragma unroll
    for (int qi = 0; qi < NQ; ++qi) {
        float* zq = sp<float>(zs_base + qi * ZQ * 4);
        float m = -INFINITY;
#pragma unroll 1
        for (int jj = lane; jj < n; jj += 32) m = fmaxf(m, zq[jj]);
        m = warp_max(m);
        float s = 0.f;
#pragma unroll 1
        for (int jj = lane; jj < n; jj += 32) { const float e = exp2f(zq[jj] - m); zq[jj] = e; s += e; }
        s = warp_sum(s);
        mq[qi] = m; sq[qi] = s;
    }
    if (hdr.sync) {
        if (lane == 0) {
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) { ms[(u * kXq + qi) * 2] = mq[qi]; ms[(u * kXq + qi) * 2 + 1] = sq[qi]; }
        }
        if (!team_sync()) return false;
        const int u0 = u - d.span;
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) {
            float M = -INFINITY;
            for (int s = 0; s < spr; ++s) M = fmaxf(M, ms[((u0 + s) * kXq + qi) * 2]);
            float tot = 0.f;
            for (int s = 0; s < spr; ++s) tot += ms[((u0 + s) * kXq + qi) * 2 + 1] * exp2f(ms[((u0 + s) * kXq + qi) * 2] - M);
            sq[qi] = exp2f(mq[qi] - M) / tot;
        }
    } else {
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) sq[qi] = 1.0f / sq[qi];
    }
    __syncwarp();
#pragma unroll
    for (int qi = 0; qi < NQ; ++qi) {
        float* zq = sp<float>(zs_base + qi * ZQ * 4);
        unsigned short* zh = reinterpret_cast<unsigned short*>(zq);
        float* Srow = (S_base && (qi % NQI) < nq) ? S_base + (qi / NQI) * S_hstride + (qi % NQI) * S_qstride : nullptr;
        const float inv = sq[qi];
#pragma unroll 1
        for (int j0 = 0; j0 < n_pad; j0 += 32) {      // warp-uniform trip count
            const int jj = j0 + lane;
            const float w = jj < n ? zq[jj] * inv : 0.f;
            if (Srow && jj < n) Srow[jj] = w;
            __syncwarp();
            if (jj < n_pad) {
                const __nv_bfloat16 hi = __float2bfloat16_rn(w);
                const __nv_bfloat16 lo = __float2bfloat16_rn(w - __bfloat162float(hi));
                const int at = packed_slot(jj);
                zh[at] = *reinterpret_cast<const unsigned short*>(&hi);
                if (kWeightRemainder) zh[at + 4] = *reinterpret_cast<const unsigned short*>(&lo);
            }
        }
    }
    __syncwarp();
    return true;
}

// The outputs of one layer and one head from the accumulators: acc[x][0], [1] hold dim 16x + gid
// of queries 2tig, 2tig+1 and acc[x][2], [3] dim 16x + gid + 8.  They are rounded to bf16 into
// the warp's scratch rows (the query rows there are no longer needed), row = query * R + head, so
// that the heads of one query lie side by side as they do in the output.
template <int NQ>
__device__ __forceinline__ void StepConsumer::stage_rows(const float (&acc)[4][4], int nq, int R, int hh) {
    const int tig = lane & 3, gid = lane >> 2;
    __nv_bfloat16* stage = sp<__nv_bfloat16>(scr_off);
    if (NQ == 1) {
        if (tig == 0) {
#pragma unroll
            for (int x = 0; x < 4; ++x) { stage[hh * kDh + 16 * x + gid] = __float2bfloat16_rn(acc[x][0]); stage[hh * kDh + 16 * x + gid + 8] = __float2bfloat16_rn(acc[x][2]); }
        }
    } else {
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            if (2 * tig < nq) {
                stage[((2 * tig) * R + hh) * kDh + 16 * x + gid] = __float2bfloat16_rn(acc[x][0]);
                stage[((2 * tig) * R + hh) * kDh + 16 * x + gid + 8] = __float2bfloat16_rn(acc[x][2]);
            }
            if (2 * tig + 1 < nq) {
                stage[((2 * tig + 1) * R + hh) * kDh + 16 * x + gid] = __float2bfloat16_rn(acc[x][1]);
                stage[((2 * tig + 1) * R + hh) * kDh + 16 * x + gid + 8] = __float2bfloat16_rn(acc[x][3]);
            }
        }
    }
}
// The staged rows of a layer to the output, 16 bytes per lane: piece i = (query, head, chunk).
__device__ __forceinline__ void StepConsumer::flush_rows(char* orow, int nq, int R, long long O_qstride) {
    __syncwarp();
    const int pieces = nq * R * 8;
    for (int i = lane; i < pieces; i += 32) {
        const int row = i >> 3, c = i & 7;
        const int qi = R == 4 ? row >> 2 : R == 2 ? row >> 1 : row, hh = row - qi * R;
        *reinterpret_cast<uint4*>(orow + qi * O_qstride + hh * 128 + c * 16) = *sp<uint4>(scr_off + row * 128 + c * 16);
    }
    __syncwarp();
}

// One attention unit on the tensor cores: R rows (heads) of one (block, id) side by side inside
// each phase, so that what a unit costs beside its arithmetic (descriptors, barrier waits,
// address set-up, output stores) is paid once for all of them and the heads' independent chains
// of loads and MMAs overlap.
//   scores:  D[16 positions x 8 queries] = K_tile[16 x 64] . q^T              (queries padded to 8)
//   apply:   D[16 dims x 8 queries]     += V_tile^T[16 x 16 positions] . S^T   (four dim tiles)
// S is applied as bf16; products and sums are float32.  Columns of D that belong to padding
// queries are computed from whatever the padding lanes load and are never stored.
template <int NQ, int R>
__device__ void StepConsumer::attend(const UnitDesc& d, const BundleHdr& hdr) {
    const TeamKind& kp = p.k[d.kind];
    const int ZQ = (int)kp.zq;
    const int n = d.n, nq = d.nq, pi = d.pi, tp = d.tp, new_row = d.new_row;
    const int my_tiles = (n + tp - 1) / tp;
    const int tig = lane & 3, gid = lane >> 2;                 // mma fragment coordinates
    const long long layer_bytes = kp.layer_bytes;
    const unsigned panel_bytes = kp.panel_bytes;
    const uint32_t zs_head = (uint32_t)(NQ * ZQ * 4);          // bytes between the score rows of two heads

    // ---- this unit's small rows, fetched by the warp itself while the producer's copies are in
    // flight.  Scratch rows: [qi * R + hh] = query qi of head hh; then R rows = this step's key
    // rows; then [l * R + hh] = this step's value rows of layer l (the last two groups only when
    // the span ends in the new position).
    const int scr_k = nq * R, scr_v = scr_k + R;
    {
        const int rows = scr_k + (new_row >= 0 ? R * (1 + pi) : 0);
        const unsigned q_stride = (unsigned)p.H * 128u;
        for (int i = lane; i < rows * 8; i += 32) {
            const int row = i >> 3, c = i & 7;
            const char* src;
            if (row < scr_k) { const int qi = row / R; src = d.q + (unsigned long long)qi * q_stride + (row - qi * R) * 128; }
            else if (row < scr_v) src = d.knew + (row - scr_k) * 128;
            else { const int lr = row - scr_v, l = lr / R; src = d.vnew + (long long)l * layer_bytes + (lr - l * R) * 128; }
            cp_async16(sm.sm_base + scr_off + row * 128 + c * 16, src + c * 16);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    }

    // ldmatrix: this lane addresses row lrow of a 16-row block and, for the pair of 16-byte
    // chunks 2x, 2x+1, the chunk 2x + (lane >> 4).  Cached rows keep chunk c at c ^ (row & 7)
    // (row & 7 == lane & 7 here).  This step's own row is not in the tile: the lane that addresses
    // its position reads it from the warp's scratch rows instead, where it lies in natural order
    // (new_fix takes the permutation out again).
    const int lrow = (lane & 7) + ((lane >> 3) & 1) * 8;
    const uint32_t new_fix = (uint32_t)(lane & 7) << 4;
    uint32_t ld_swz[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) ld_swz[x] = (uint32_t)(((2 * x + (lane >> 4)) ^ (lane & 7)) << 4);
    const uint32_t scr_s = sm.sm_base + scr_off;

    // ---- key tiles: scores into the warp's score slots (log2 domain)
    const float sc = p.scale_log2e;
    const uint32_t zk = zs_off + ((2 * tig) * ZQ + gid) * 4;   // queries 2tig, 2tig+1; positions gid, gid+8
    for (int t = 0; t < hdr.tiles; ++t) {
        const int slot = acquire();
        if (slot < 0) return;
        if (t == 0) {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncwarp();
        }
        if (t < my_tiles) {
            const uint32_t st0 = my_rows(slot);
            const int s0 = t * tp;
            const int r = min(tp, n - s0);
            const int nr = (new_row >= s0 && new_row < s0 + r) ? new_row - s0 : -1;   // this step's key row in the tile
            // every head's query rows (natural chunk order) as B fragments (k = dims, n = query)
            uint32_t qb[R][4][2];
#pragma unroll
            for (int hh = 0; hh < R; ++hh) {
                const uint32_t qrow = scr_off + (uint32_t)((gid < nq ? gid : 0) * R + hh) * 128u + 4u * tig;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    qb[hh][ks][0] = *sp<uint32_t>(qrow + 32 * ks);
                    qb[hh][ks][1] = *sp<uint32_t>(qrow + 32 * ks + 16);
                }
            }
            if (nr >= 0 && d.dstK && lane < 8 * R) {                                  // into the cache, chunk-permuted
                const int hh = lane >> 3, c = lane & 7;
                *reinterpret_cast<uint4*>(d.dstK + (unsigned long long)hh * panel_bytes + ((c ^ (nr & 7)) << 4)) =
                    *sp<uint4>(scr_off + (scr_k + hh) * 128 + c * 16);
            }
            const uint32_t st_s = sm.sm_base + st0 + (uint32_t)lrow * 128u;
            const uint32_t head_bytes = (uint32_t)r * 128u;                          // a head's rows follow the previous head's
#pragma unroll 1
            for (int b0 = 0; b0 < r; b0 += 16) {
                const bool is_new = (b0 + lrow == nr);
                const uint32_t fix = is_new ? new_fix : 0u;
                float acc[R][4];
                uint32_t a[R][4][4];
#pragma unroll
                for (int hh = 0; hh < R; ++hh) {
                    const uint32_t rb = is_new ? scr_s + (scr_k + hh) * 128 : st_s + hh * head_bytes + b0 * 128;
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) ldsm_x4(rb + (ld_swz[ks] ^ fix), a[hh][ks]);
                }
#pragma unroll
                for (int hh = 0; hh < R; ++hh) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[hh][e] = 0.f;
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) mma_bf16(acc[hh], a[hh][ks][0], a[hh][ks][1], a[hh][ks][2], a[hh][ks][3], qb[hh][ks][0], qb[hh][ks][1]);
                }
                // acc[0], acc[1]: position b0+gid, queries 2tig, 2tig+1; acc[2], acc[3]: position b0+gid+8.
                // Rows of the block at or beyond r (another head's or unit's rows, stale bytes) give
                // scores that are never stored.
                const int pos = s0 + b0 + gid;
#pragma unroll
                for (int hh = 0; hh < R; ++hh) {
                    float* z = sp<float>(zk + hh * zs_head + (s0 + b0) * 4);
                    if (2 * tig < NQ) {
                        if (pos < n) z[0] = acc[hh][0] * sc;
                        if (pos + 8 < n) z[8] = acc[hh][2] * sc;
                    }
                    if (2 * tig + 1 < NQ) {
                        if (pos < n) z[ZQ] = acc[hh][1] * sc;
                        if (pos + 8 < n) z[ZQ + 8] = acc[hh][3] * sc;
                    }
                }
            }
        }
        release();
    }
    __syncwarp();

    const int n_pad = (n + 15) & ~15;
    if (!softmax<R * NQ, NQ>(d, hdr, n, n_pad, ZQ, zs_off, d.S, kp.S_ld, (long long)p.H * kp.S_ld, nq)) return;

    // ---- value tiles, layer by layer
    // B fragments: the weights of query gid at positions b0 + {2tig, 2tig+1} and b0 + {2tig+8, 2tig+9},
    // one load per block straight from the packed words.
    // A fragments: the tile transposed by ldmatrix; this lane addresses position vrow of a block
    // and, for the dim tile x, the 16-byte chunk 2x + ((lane >> 3) & 1).
    const uint32_t za = zs_off + (gid < NQ ? gid : 0) * ZQ * 4 + tig * 16;
    const int vrow = (lane & 7) + ((lane >> 4) << 3);
    uint32_t vd_swz[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) vd_swz[x] = (uint32_t)(((2 * x + ((lane >> 3) & 1)) ^ (lane & 7)) << 4);
    const long long plane_bytes = kp.plane_bytes;
    char* vlast = d.dstV;                                             // where this step's value row goes
    const long long O_qstride = (long long)p.H * 128;
    char* op = d.O;
    const int spr = 1 << d.spr_log2;
#pragma unroll 1
    for (int l = 0; l < hdr.layers; ++l) {
        // Several heads: each is one tile (the host cuts them so) and is done inside it.  A lone head
        // keeps its sums across the tiles of the layer.
        float acc[R][4][4];
#pragma unroll
        for (int hh = 0; hh < R; ++hh)
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[hh][x][e] = 0.f;
#pragma unroll 1
        for (int t = 0; t < hdr.tiles; ++t) {
            const int slot = acquire();
            if (slot < 0) return;
            if (l < pi && t < my_tiles) {
                const uint32_t st0 = my_rows(slot);
                const int s0 = t * tp;
                const int r = min(tp, n - s0);
                const int nr = (new_row >= s0 && new_row < s0 + r) ? new_row - s0 : -1;
                if (nr >= 0 && lane < 8 * R) {
                    const int hh = lane >> 3, c = lane & 7;
                    *reinterpret_cast<uint4*>(vlast + (unsigned long long)hh * panel_bytes + ((c ^ (nr & 7)) << 4)) =
                        *sp<uint4>(scr_off + (scr_v + l * R + hh) * 128 + c * 16);
                }
                const uint32_t st_s = sm.sm_base + st0 + (uint32_t)vrow * 128u;
                const uint32_t head_bytes = (uint32_t)r * 128u;
#pragma unroll 1
                for (int b0 = 0; b0 < r; b0 += 16) {
                    // rows at or beyond r hold other bytes: their weights are zero, but 0 x NaN would not be,
                    // so those lanes address a row of zeros instead
                    const int row = b0 + vrow;
                    const bool is_new = (row == nr);
                    const uint32_t fix = is_new ? new_fix : 0u;
                    uint2 w[R];                                          // (weights of b0.., weights of b0+8..) per head
                    uint32_t a[R][4][4];
#pragma unroll
                    for (int hh = 0; hh < R; ++hh) {
                        w[hh] = *sp<uint2>(za + hh * zs_head + (s0 + b0) * 4);
                        const uint32_t rb = is_new ? scr_s + (scr_v + l * R + hh) * 128 : st_s + hh * head_bytes + b0 * 128;
#pragma unroll
                        for (int x = 0; x < 4; ++x) ldsm_x4_t(row >= r ? zero_row : rb + (vd_swz[x] ^ fix), a[hh][x]);
                    }
#pragma unroll
                    for (int hh = 0; hh < R; ++hh)
#pragma unroll
                        for (int x = 0; x < 4; ++x) mma_bf16(acc[hh][x], a[hh][x][0], a[hh][x][1], a[hh][x][2], a[hh][x][3], w[hh].x, w[hh].y);
                }
            }
            release();
        }
        // acc[hh][x][0], [1]: dim 16x + gid of queries 2tig, 2tig+1; [2], [3]: dim 16x + gid + 8
        bool store = l < pi;
        if (hdr.sync) {
            // the spans of a row add up their partial outputs through shared memory (two buffers, by layer parity)
            float* xo = sp<float>(xch_o(l & 1));
            if (l < pi && spr > 1) {
                float* mine = xo + u * p.xo_unit_floats + (2 * tig) * kDh + gid;
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (2 * tig < NQ) mine[16 * x + 8 * h] = acc[0][x][2 * h];
                        if (2 * tig + 1 < NQ) mine[kDh + 16 * x + 8 * h] = acc[0][x][2 * h + 1];
                    }
            }
            if (!team_sync()) return;
            if (l < pi && spr > 1) {
                store = false;
                if (d.span == 0) {
                    char* orow = op + lane * 4;
                    for (int qi = 0; qi < nq; ++qi) {
                        float2 s2 = make_float2(0.f, 0.f);
                        for (int s = 0; s < spr; ++s) {
                            const float2 v = *reinterpret_cast<const float2*>(xo + (u + s) * p.xo_unit_floats + qi * kDh + 2 * lane);
                            s2.x += v.x; s2.y += v.y;
                        }
                        *reinterpret_cast<uint32_t*>(orow + qi * O_qstride) = pack_bf16x2(s2.x, s2.y);
                    }
                }
            }
        }
        if (store) {
#pragma unroll
            for (int hh = 0; hh < R; ++hh) stage_rows<NQ>(acc[hh], nq, R, hh);
            flush_rows(op, nq, R, O_qstride);
        }
        if (vlast) vlast += plane_bytes;
        op += layer_bytes;
    }
}

template <int NQE>
__global__ void __launch_bounds__(kStepWarps * 32, 1) decode_step_team_kernel(const __grid_constant__ TeamParams p) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // The launch allows programmatic stream serialization (see decode_step_kernel): only the
    // set-up of shared memory runs ahead of the preceding kernel's completion.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    StepSmem sm;
    sm.sm_base = smem_u32(san_smem); sm.off_desc = p.off_desc; sm.off_bars = p.off_bars;
    if (threadIdx.x < 32) *sp<uint32_t>(p.off_zero + threadIdx.x * 4) = 0u;
    if (threadIdx.x == 0) {
        for (int t = 0; t < kTeams; ++t) {
            for (int s = 0; s < kNS; ++s) {
                mbar_init(sp<uint64_t>(p.off_bars + t * kTeamBarBytes + s * 8), 1);
                mbar_init(sp<uint64_t>(p.off_bars + t * kTeamBarBytes + (kNS + s) * 8), kTeamWarps);
            }
            for (int s = 0; s < kNS; ++s) mbar_init(sp<uint64_t>(p.off_bars + t * kTeamBarBytes + (2 * kNS + s) * 8), 1);
            mbar_init(sp<uint64_t>(p.off_bars + t * kTeamBarBytes + 3 * kNS * 8), kTeamWarps);
        }
        *sm.dead_flag() = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp >= kStepConsumers) {
        // ------------------------------------------------------------------ a team's producer warp
        StepProducer pr(p);
        pr.sm = sm; pr.lane = lane; pr.team = warp - kStepConsumers;
        pr.ring0 = (uint32_t)pr.team * p.ring_stride;
        pr.head_v = pr.tail_v = pr.head_p = 0; pr.n_slots = pr.n_retired = pr.n_bundles = 0; pr.dead = false;
        pr.rec_end_v = 0;
        const int team = pr.team;
        const unsigned S = 1u << max(p.k[0].spr_log2, p.k[1].spr_log2);      // bundles start and end on whole rows
        auto chunk_for = [&](unsigned start) -> unsigned {
            const unsigned left = start < p.n_units ? p.n_units - start : 0u;
            unsigned c = left / p.grab_teams;
            c &= ~(S - 1u);
            return min((unsigned)kTeamWarps, max(S, c));
        };
        // Every team's first bundle is fixed by its place in the grid (no round trip to the counter
        // before the first copy can go out); the counter hands out the units after those.
        const unsigned dyn0 = (unsigned)gridDim.x * kTeams * kTeamWarps;
        auto grab = [&](unsigned chunk) -> unsigned {
            unsigned v = 0;
            if (lane == 0) v = dyn0 + (unsigned)atomicAdd(p.queue, (int)chunk);
            return v;
        };
        // Two bundles are in preparation behind the one being issued: the index of the one after
        // next is on its way back from the counter, the id / length entries of the next one are
        // on their way from memory.
        unsigned cur_chunk = kTeamWarps;
        unsigned cur = ((unsigned)blockIdx.x * kTeams + (unsigned)team) * kTeamWarps;
        unsigned nxt_chunk = chunk_for(dyn0);
        const unsigned nxt_raw0 = grab(nxt_chunk);
        // Lane u * kUnitRows + hh works for head hh of the bundle's unit u: the lanes of a unit decode
        // it alike, each issues the copy of its own head's rows.
        constexpr int kCopyLanes = kTeamWarps * kUnitRows;
        const int lu = lane / kUnitRows, hh = lane % kUnitRows;
        UnitIdx cur_ui;
        unit_index(p, cur + (unsigned)lu, lu < (int)cur_chunk, &cur_ui);
        unsigned nxt = __shfl_sync(0xffffffffu, nxt_raw0, 0);
        while (cur < p.n_units && !pr.dead) {
            const unsigned aft_chunk = chunk_for(nxt);
            const unsigned aft_raw = grab(aft_chunk);                          // used at the end of the iteration
            UnitIdx nxt_ui;
            unit_index(p, nxt + (unsigned)lu, lu < (int)nxt_chunk, &nxt_ui);
            pr.ensure_slot();
            if (pr.dead) break;
            const int bslot = (int)(pr.n_bundles % kNS);
            ProdUnit pu;
            UnitDesc ud;
            decode_unit(p, cur_ui, hh == 0, &pu, &ud);
            // the bundle: tiles per plane, value layers, whether any row is split over spans
            int tiles = pu.tiles, layers = pu.pi, sync = pu.spr_log2;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                tiles = max(tiles, __shfl_xor_sync(0xffffffffu, tiles, o));
                layers = max(layers, __shfl_xor_sync(0xffffffffu, layers, o));
                sync = max(sync, __shfl_xor_sync(0xffffffffu, sync, o));
            }
            tiles = max(tiles, 1);
            if (lane == 0) *sp<BundleHdr>(sm.bundle_hdr(team, bslot)) = BundleHdr{tiles, layers, sync ? 1 : 0, 0};
            if (hh == 0 && lu < kTeamWarps) *sp<UnitDesc>(sm.unit_desc(team, bslot, lu)) = ud;
            __syncwarp();
            if (lane == 0) mbar_arrive(sm.bar_ready(team, bslot));     // the consumers may start on their small rows
            // ---- slots: the key tiles, then each layer's value tiles
            const bool attn = lane < kCopyLanes && (pu.kind == UK_SELF || pu.kind == UK_ENC);
            for (int plane = 0; plane <= layers && !pr.dead; ++plane) {
                for (int t = 0; t < tiles && !pr.dead; ++t) {
                    const int r = (attn && plane <= pu.pi && t < pu.tiles) ? min(pu.tp, pu.n - t * pu.tp) : 0;   // rows of one head
                    // rows of the units before this one (a unit's lanes agree; only lanes hh == 0 are added up)
                    int off = (hh == 0) ? r * pu.rows : 0;
#pragma unroll
                    for (int o = kUnitRows; o < kCopyLanes; o <<= 1) {
                        const int a = __shfl_up_sync(0xffffffffu, off, o);
                        if (lane >= o) off += a;
                    }
                    const int tot = __shfl_sync(0xffffffffu, off, kCopyLanes - kUnitRows);
                    off = __shfl_sync(0xffffffffu, off, lu * kUnitRows) - r * pu.rows;
                    const uint32_t bytes = (uint32_t)tot * 128u;
                    pr.ensure_slot();
                    const uint32_t base = pr.alloc(bytes);
                    if (pr.dead) break;
                    const int slot = (int)(pr.n_slots % kNS);
                    const uint32_t sd = sm.slot_desc(team, slot);
                    if (lane == 0) *sp<uint32_t>(sd) = base;
                    if (hh == 0 && lu < kTeamWarps) *sp<uint16_t>(sd + 4 + 2 * lu) = (uint16_t)off;
                    // this step's row is not cached yet: the consumer reads it from its own scratch rows
                    const bool copies = r > 0 && hh < pu.rows;
                    const bool with_new = copies && pu.new_row >= t * pu.tp && pu.new_row < t * pu.tp + r;
                    const uint32_t cached = copies ? (uint32_t)(r - (with_new ? 1 : 0)) * 128u : 0u;
                    uint32_t tx = cached;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) tx += __shfl_xor_sync(0xffffffffu, tx, o);
                    __syncwarp();
                    const uint32_t bar = sm.bar_full(team, slot);
                    if (lane == 0) mbar_expect_tx(bar, tx);
                    if (cached) {
                        const char* src = (plane == 0 ? pu.srcK : pu.srcV + (long long)(plane - 1) * pu.plane_bytes) +
                                          (unsigned long long)hh * pu.panel_bytes + (unsigned)(t * pu.tp) * 128u;
                        bulk_g2s(sm.sm_base + base + (uint32_t)(off + hh * r) * 128u, src, cached, bar);
                    }
                    pr.issued();
                }
            }
            pr.n_bundles += 1;
            cur = nxt; cur_chunk = nxt_chunk; cur_ui = nxt_ui;
            nxt = __shfl_sync(0xffffffffu, aft_raw, 0); nxt_chunk = aft_chunk;
        }
        // ---- no more work: tell the team, then leave the counters clean for the next launch
        if (!pr.dead) pr.ensure_slot();
        if (!pr.dead) {
            if (lane == 0) {
                *sp<BundleHdr>(sm.bundle_hdr(team, (int)(pr.n_bundles % kNS))) = BundleHdr{0, 0, 0, 1};
                mbar_arrive(sm.bar_ready(team, (int)(pr.n_bundles % kNS)));
            }
        } else {
            // a wait ran out somewhere: let the copies already issued land before the CTA leaves
            for (uint32_t s = pr.n_retired; s != pr.n_slots; ++s) {
                const uint32_t bar = sm.bar_full(team, (int)(s % kNS));
                const long long t0 = clock64();
                while (!mbar_try_wait(bar, (s / kNS) & 1u) && clock64() - t0 < 200000000LL) {}
            }
        }
        if (lane == 0) {
            __threadfence();
            const int done = atomicAdd(p.queue + 1, 1);
            if (done == (int)gridDim.x * kTeams - 1) { p.queue[0] = 0; p.queue[1] = 0; __threadfence(); }
        }
        return;
    }

    // ---------------------------------------------------------------------- consumer warps
    StepConsumer c(p);
    c.sm = sm; c.lane = lane; c.team = warp / kTeamWarps; c.u = warp % kTeamWarps;
    c.cs = 0; c.xs = 0; c.dead = false;
    c.zs_off = p.off_zs + (uint32_t)warp * p.zs_bytes;
    c.scr_off = p.off_scr + (uint32_t)warp * p.scr_bytes;
    c.zero_row = sm.sm_base + p.off_zero;
    for (uint32_t b = 0; !c.dead; ++b) {
        const int bslot = (int)(b % kNS);
        {
            const uint32_t bar = sm.bar_ready(c.team, bslot), par = (b / kNS) & 1u;
            if (!mbar_try_wait(bar, par) && !step_wait_slow(bar, par, sm.dead_flag())) { c.fail(4); break; }
        }
        const BundleHdr hdr = *sp<BundleHdr>(sm.bundle_hdr(c.team, bslot));
        if (hdr.end) break;
        const UnitDesc d = *sp<UnitDesc>(sm.unit_desc(c.team, bslot, c.u));
        if (d.kind == UK_AAN) c.aan(d);
        if (d.kind == UK_ENC && NQE > 1) {
            if (d.rows == 2) c.template attend<NQE, 2>(d, hdr); else c.template attend<NQE, 1>(d, hdr);
        } else if (d.kind == UK_SELF || d.kind == UK_ENC) {
            if (d.rows == 4) c.template attend<1, 4>(d, hdr); else if (d.rows == 2) c.template attend<1, 2>(d, hdr); else c.template attend<1, 1>(d, hdr);
        } else {
            c.idle(hdr);
        }
    }
}

}  // namespace san
