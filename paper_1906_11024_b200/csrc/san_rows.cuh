// One decode step in one launch for sentence-sized rows (every row at most kRowsMaxPos
// positions, bf16): cache append, weights (Eq. 1) and apply (Eq. 2 with Eq. 4) for every block
// of both attention kinds, plus the AAN running average.
//
// The list of work items, their decoding and their hand-out to the warps of a CTA are those of
// decode_step_kernel.  What differs is how a warp works through an item, because with rows this
// short a step is as long as the chain of dependent instructions and memory round trips of the
// items one warp takes one after the other:
//   * a whole plane of an item (its key rows, or the value rows of one layer) is one copy and one
//     barrier, and the planes of the next items are requested while the warp still computes on
//     this one: each warp owns a ring of kRowsRing bytes that holds planes of any size back to
//     back.  All planes that fit are requested by ONE copy instruction, lane j issuing the j-th
//     of them (a bulk copy costs its warp about 400 cycles to issue whatever its size, 55 more
//     for each further lane);
//   * the query rows and this step's own key / value rows (not yet in the cache) are fetched in
//     16-byte pieces (cp.async) into the plane's slot, the latter already chunk-permuted like a
//     cached row, so that the arithmetic sees one uniform tile;
//   * the queries are the M side of the tensor-core products (16 rows, 1 to 8 of them real):
//       scores:  D[16 queries x 8 positions] = q[16 x 64] . K_tile^T
//       apply:   D[16 queries x 8 dims]     += S[16 x 16 positions] . V_tile
//     so the accumulators of the first product, once normalised in registers (a row's maximum
//     and sum take two shuffles), are the A fragments of the second: scores never go through
//     shared memory, and everything is unrolled for the item's number of 16-position blocks.
// S is applied as bf16; products and sums are float32.
#pragma once

#include "san_fused.cuh"

namespace san {

constexpr int kRowsWarps = 16;
constexpr int kRowsRing = 13312;        // bytes per warp: 104 rows
constexpr int kRowsSlots = 8;           // planes in flight per warp at most (one barrier each)
constexpr int kRowsMaxBlocks = 6;
constexpr int kRowsMaxPos = 16 * kRowsMaxBlocks;   // positions per row at most; a key plane with 8 query rows still fits the ring
static_assert((kRowsMaxPos + 8) * 128 <= kRowsRing, "a key plane and its query rows fit the ring");

enum { TAG_ROWS = 9 };
constexpr bool kRowsKernelByDefault = false;

constexpr size_t rows_smem_bytes() {
    return (size_t)kRowsWarps * (kRowsRing + kRowsSlots * sizeof(uint64_t)) + 128 /* a row of zeros */ + (size_t)kCtaItems * sizeof(ItemDesc);
}

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// D(16x8) += A(16x16) * B(16x8) where rows 8..15 of A are zero.  d[2], d[3] (rows 8..15 of D) stay
// zero; they are carried along because the instruction takes its accumulator as four registers in a row.
__device__ __forceinline__ void mma_bf16_top(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%5}, {%7,%8}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(0u), "r"(a2), "r"(b0), "r"(b1));
}

struct RowWarp {
    const StepParams& p;
    uint32_t sm_base;             // shared-space address of san_smem
    uint32_t ring, bars;          // offsets of this warp's ring and of its barriers
    uint32_t descs_off;           // offset of the CTA's decoded items
    uint32_t zero_row;            // shared-space address of 128 zero bytes
    unsigned* q_next;             // shared counter: next item to hand out
    unsigned n_valid;
    int lane;
    // copy side: the item whose planes are being requested, and the one after (taken ahead)
    bool p_active;
    unsigned p_idx, nx_idx;
    int p_plane;                  // 0 = keys, l + 1 = values of the item's layer l
    uint32_t head_v, tail_v, head_p;   // ring: virtual byte counters of what was requested / given back, physical write offset
    uint32_t n_slots, n_ret;      // planes requested / given back
    uint32_t rec_base, rec_end;   // lane i: offset of the plane with sequence number i (mod kRowsSlots), head_v behind it,
    uint32_t rec_grp;             //         and the cp.async group its small rows went out with
    uint32_t n_groups;            // cp.async groups committed so far (one per top_up that requested anything)
    unsigned long long fifo;      // items whose planes are (being) requested and whose arithmetic is still to do
    int fifo_n;
    bool dead;                    // a wait ran out: leave

    __device__ RowWarp(const StepParams& pp) : p(pp) {}

    __device__ __forceinline__ const ItemDesc& desc(unsigned idx) const {
        return *sp<ItemDesc>(descs_off + idx * (uint32_t)sizeof(ItemDesc));
    }
    __device__ __forceinline__ unsigned grab() {
        unsigned k = 0;
        if (lane == 0) k = atomicAdd(q_next, 1u);
        return __shfl_sync(0xffffffffu, k, 0);
    }
    __device__ __forceinline__ void next_item() {
        p_idx = nx_idx;
        p_active = p_idx < n_valid;
        if (!p_active) return;
        fifo |= (unsigned long long)p_idx << (8 * fifo_n);
        fifo_n += 1;
        nx_idx = grab();
        p_plane = 0;
    }
    __device__ __forceinline__ void fail(int where) {
        if (lane == 0 && atomicCAS(&p.err[0], 0, (int)SAN_ERR_TIMEOUT) == 0) { p.err[1] = TAG_ROWS; p.err[2] = where; }
        dead = true;
    }

    // Requests, in order, as many of the planes still to come as the ring and its barriers have room
    // for: ONE copy instruction, lane j issuing the j-th of them.  The planes of an item lie back to
    // back (key rows, query rows, then each layer's value rows), so every lane works out its own
    // plane's place without a loop over planes.
    __device__ __forceinline__ void top_up() {
        uint32_t my_dst = 0, my_bytes = 0, my_bar = 0;
        const char* my_src = nullptr;
        int k = 0;                                   // planes requested so far in this call (lanes 0 .. k-1)
        while (p_active) {
            const int room = kRowsSlots - (int)(n_slots - n_ret);
            if (room == 0) break;
            const ItemDesc& d = desc(p_idx);
            const int n = d.n, has_new = d.has_new, nq = d.nq, pi = d.pi;
            const uint32_t S = (uint32_t)n * 128u, Q = p_plane == 0 ? (uint32_t)nq * 128u : 0u;
            const int want = min(pi + 1 - p_plane, room);
            // how many of them fit in one piece: behind head_p, else from the start of the ring
            uint32_t hv = head_v, hp = head_p;
            const uint32_t free_all = (uint32_t)kRowsRing - (hv - tail_v), run = (uint32_t)kRowsRing - hp;
            const uint32_t need_me = Q + (uint32_t)(lane + 1) * S;      // bytes of the first lane + 1 planes
            int m = __popc(__ballot_sync(0xffffffffu, lane < want && need_me <= min(run, free_all)));
            if (m == 0) {
                if (free_all <= run) break;
                m = __popc(__ballot_sync(0xffffffffu, lane < want && need_me <= free_all - run));
                if (m == 0) break;
                hv += run; hp = 0;
            }
            const uint32_t base = ring + hp;
            const KindParams& kp = p.k[d.kind];
            const int j = lane - k;
            if (j >= 0 && j < m) {
                const int pl = p_plane + j;
                my_dst = sm_base + base + (uint32_t)j * S + (j > 0 ? Q : 0u);
                my_src = pl == 0 ? d.srcK : d.srcV + (long long)(pl - 1) * kp.plane_bytes;
                my_bytes = (uint32_t)(n - has_new) * 128u;
                my_bar = sm_base + bars + ((n_slots + (uint32_t)j) % kRowsSlots) * 8u;
            }
            {   // lane L < kRowsSlots keeps the record of the plane with sequence number L (mod kRowsSlots)
                const uint32_t jj = ((uint32_t)lane - n_slots) % kRowsSlots;
                if (lane < kRowsSlots && jj < (uint32_t)m) {
                    rec_base = base + jj * S + (jj > 0 ? Q : 0u);
                    rec_end = hv + Q + (jj + 1) * S;
                    rec_grp = n_groups;
                }
            }
            if (has_new) {      // this step's row closes every plane, chunk-permuted like a cached row: 8 lanes per plane
                const int c = lane & 7;
                for (int j2 = lane >> 3; j2 < m; j2 += 4) {
                    const int pl = p_plane + j2;
                    const char* nw = pl == 0 ? d.knew : d.vnew + (long long)(pl - 1) * kp.layer_bytes;
                    cp_async_16(sm_base + base + (uint32_t)j2 * S + (j2 > 0 ? Q : 0u) + (uint32_t)(n - 1) * 128u + (uint32_t)((c ^ ((n - 1) & 7)) << 4), nw + c * 16);
                }
            }
            if (p_plane == 0) {             // the query rows ride behind the key rows: chunk c of row r at c ^ r
                const unsigned q_stride = (unsigned)p.H * 128u;
                for (int i = lane; i < nq * 8; i += 32) {
                    const int r = i >> 3, c = i & 7;
                    cp_async_16(sm_base + base + S + (uint32_t)r * 128u + (uint32_t)((c ^ r) << 4), d.q + (unsigned long long)r * q_stride + c * 16);
                }
            }
            const uint32_t tot = Q + (uint32_t)m * S;
            head_v = hv + tot; head_p = hp + tot;
            n_slots += (uint32_t)m; k += m;
            p_plane += m;
            if (p_plane > pi) next_item(); else break;      // no room for the rest of this item yet
        }
        if (k == 0) return;
        asm volatile("cp.async.commit_group;" ::: "memory");
        n_groups += 1;
        if (lane < k) {
            mbar_expect_tx(my_bar, my_bytes);
            if (my_bytes) bulk_g2s(my_dst, my_src, my_bytes, my_bar);
        }
    }

    // Waits for the next plane in order; returns the offset of its rows, or kNoPlane after a timeout.
    static constexpr uint32_t kNoPlane = 0xffffffffu;
    __device__ __forceinline__ uint32_t acquire() {
        if (n_ret == n_slots) { fail(100); return kNoPlane; }      // top_up always finds room in an empty ring
        const uint32_t seq = n_ret;
        const uint32_t bar = sm_base + bars + (seq % kRowsSlots) * 8u, par = (seq / kRowsSlots) & 1u;
        if (!mbar_try_wait(bar, par) && !mbar_wait_slow(bar, par)) { fail((int)(seq % kRowsSlots)); return kNoPlane; }
        // The plane's small rows: groups complete in order, and all but the latest have had an item's
        // worth of arithmetic to arrive, so only a plane requested by the latest top_up waits for that one too.
        const uint32_t grp = __shfl_sync(0xffffffffu, rec_grp, (int)(seq % kRowsSlots));
        if (grp + 1 == n_groups) asm volatile("cp.async.wait_group 0;" ::: "memory");
        else asm volatile("cp.async.wait_group 1;" ::: "memory");
        __syncwarp();
        return __shfl_sync(0xffffffffu, rec_base, (int)(seq % kRowsSlots));
    }
    // Every lane is done with the plane: its bytes and its barrier are free again.
    __device__ __forceinline__ void release() {
        __syncwarp();
        tail_v = __shfl_sync(0xffffffffu, rec_end, (int)(n_ret % kRowsSlots));
        n_ret += 1;
        if (n_ret == n_slots) { tail_v = head_v; head_p = 0; }      // nothing outstanding: the next plane starts the ring afresh
    }

    template <int NB> __device__ __forceinline__ void scores(const ItemDesc& d, uint32_t st, uint32_t (&pw)[2 * kRowsMaxBlocks]);
    template <int NB> __device__ __forceinline__ void apply(const ItemDesc& d, uint32_t st, const uint32_t (&pw)[2 * kRowsMaxBlocks], int l);
};

__device__ __forceinline__ float ex2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// The key plane of an item of at most NB blocks of 16 positions (at st, with the query rows behind
// the key rows): this step's key row to the cache, scores, softmax in registers, S to the caller;
// leaves the weights as bf16 pairs in pw, the A fragments of the apply products.
template <int NB>
__device__ __forceinline__ void RowWarp::scores(const ItemDesc& d, uint32_t st, uint32_t (&pw)[2 * kRowsMaxBlocks]) {
    const int n = d.n, nq = d.nq;
    const int tig = lane & 3, gid = lane >> 2;                 // mma fragment coordinates
    const int r8 = lane & 7, m4 = lane >> 3;                   // ldmatrix: this lane addresses row r8 of matrix m4
    const uint32_t st_s = sm_base + st;
    if (d.has_new && d.lead && lane < 8)                        // this step's key row into the cache (already permuted)
        *reinterpret_cast<uint4*>(const_cast<char*>(d.srcK) + (n - 1) * 128 + lane * 16) = *sp<uint4>(st + (uint32_t)(n - 1) * 128u + lane * 16);
    // A fragments of the queries: matrix m4 = rows 0..7, 16-byte chunk 4 kp + m4; registers (a0, a2) of
    // k-steps 2 kp and 2 kp + 1.  Rows 8..15 are zero and never loaded; rows at or beyond nq read zeros.
    uint32_t qa[4][2];
    {
        const uint32_t a = (r8 < nq) ? st_s + (uint32_t)(n + r8) * 128u + (uint32_t)((m4 ^ r8) << 4) : zero_row;
        const uint32_t flip = (r8 < nq) ? 64u : 0u;
        uint32_t r[4];
        ldsm_x4(a, r);        qa[0][0] = r[0]; qa[0][1] = r[1]; qa[1][0] = r[2]; qa[1][1] = r[3];
        ldsm_x4(a ^ flip, r); qa[2][0] = r[0]; qa[2][1] = r[1]; qa[3][0] = r[2]; qa[3][1] = r[3];
    }
    // B fragments of 8 positions: matrix m4 = positions 8 j + r8, chunk 4 kp + m4 (cached rows keep
    // chunk c at c ^ (position & 7)); registers (b0, b1) of k-steps 2 kp and 2 kp + 1.
    float sc[2 * NB][2];
    {
        const uint32_t ka = st_s + (uint32_t)r8 * 128u + (uint32_t)((m4 ^ r8) << 4);
#pragma unroll
        for (int j = 0; j < 2 * NB; ++j) {
            uint32_t b0[4], b1[4];
            ldsm_x4(ka + j * 1024, b0);
            ldsm_x4((ka ^ 64u) + j * 1024, b1);
            float c[4] = {0.f, 0.f, 0.f, 0.f};
            mma_bf16_top(c, qa[0][0], qa[0][1], b0[0], b0[1]);
            mma_bf16_top(c, qa[1][0], qa[1][1], b0[2], b0[3]);
            mma_bf16_top(c, qa[2][0], qa[2][1], b1[0], b1[1]);
            mma_bf16_top(c, qa[3][0], qa[3][1], b1[2], b1[3]);
            sc[j][0] = c[0]; sc[j][1] = c[1];
        }
    }
    // Softmax in registers: sc[j][e] is query gid, position 8 j + 2 tig + e (log2 domain after scaling).
    // Positions at or beyond n (the query rows, stale bytes) are masked out.
    const float scl = p.scale_log2e;
    const int lim = n - 2 * tig;                     // position 8 j + 2 tig + e is in the row iff 8 j + e < lim
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < 2 * NB; ++j)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const float v = (8 * j + e < lim) ? sc[j][e] * scl : -INFINITY;
            sc[j][e] = v;
            mx = fmaxf(mx, v);
        }
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    float sum = 0.f;
#pragma unroll
    for (int j = 0; j < 2 * NB; ++j)
#pragma unroll
        for (int e = 0; e < 2; ++e) { sc[j][e] = ex2_fast(sc[j][e] - mx); sum += sc[j][e]; }
    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
    const float inv = 1.0f / sum;
    float* Srow = (d.S && gid < nq) ? d.S + (long long)gid * ((long long)p.H * p.k[d.kind].S_ld) + 2 * tig : nullptr;
#pragma unroll
    for (int j = 0; j < 2 * NB; ++j) {
        const float w0 = sc[j][0] * inv, w1 = sc[j][1] * inv;
        if (Srow) {
            if (8 * j < lim) Srow[8 * j] = w0;
            if (8 * j + 1 < lim) Srow[8 * j + 1] = w1;
        }
        pw[j] = pack_bf16x2(w0, w1);
    }
}

// The value plane of the item's layer l (at st): this step's value row to the cache, S . V, output.
// B fragments through ldmatrix.trans: matrix m4 = positions 16 kk + 8 (m4 & 1) + r8, chunk
// 2 jp + (m4 >> 1); registers (b0, b1) of dim tiles 2 jp and 2 jp + 1.  Rows at or beyond n hold other
// bytes: their weights are zero, but 0 x NaN would not be, so those lanes address a row of zeros.
template <int NB>
__device__ __forceinline__ void RowWarp::apply(const ItemDesc& d, uint32_t st, const uint32_t (&pw)[2 * kRowsMaxBlocks], int l) {
    const int n = d.n;
    const int tig = lane & 3, gid = lane >> 2;
    const int r8 = lane & 7, m4 = lane >> 3;
    const KindParams& kp = p.k[d.kind];
    const uint32_t st_s = sm_base + st;
    if (d.has_new && lane < 8)
        *reinterpret_cast<uint4*>(const_cast<char*>(d.srcV) + (long long)l * kp.plane_bytes + (n - 1) * 128 + lane * 16) =
            *sp<uint4>(st + (uint32_t)(n - 1) * 128u + lane * 16);
    const int vpos = 8 * (m4 & 1) + r8;
    const uint32_t va = st_s + (uint32_t)vpos * 128u + (uint32_t)(((m4 >> 1) ^ r8) << 4);
    float acc[8][4];
#pragma unroll
    for (int x = 0; x < 8; ++x) { acc[x][0] = 0.f; acc[x][1] = 0.f; acc[x][2] = 0.f; acc[x][3] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < NB; ++kk) {
        const bool in_row = 16 * kk + vpos < n;
        uint32_t b[4][4];
#pragma unroll
        for (int jp = 0; jp < 4; ++jp) ldsm_x4_t(in_row ? (va + kk * 2048) ^ (uint32_t)(jp << 5) : zero_row, b[jp]);
#pragma unroll
        for (int jp = 0; jp < 4; ++jp) {
            mma_bf16_top(acc[2 * jp], pw[2 * kk], pw[2 * kk + 1], b[jp][0], b[jp][1]);
            mma_bf16_top(acc[2 * jp + 1], pw[2 * kk], pw[2 * kk + 1], b[jp][2], b[jp][3]);
        }
    }
    // acc[x][0], [1]: query gid, dims 8 x + 2 tig, + 1
    if (gid < d.nq) {
        char* op = d.O + (long long)l * kp.layer_bytes + (long long)gid * ((long long)p.H * 128) + tig * 4;
#pragma unroll
        for (int x = 0; x < 8; ++x) *reinterpret_cast<uint32_t*>(op + x * 16) = pack_bf16x2(acc[x][0], acc[x][1]);
    }
}

__global__ void __launch_bounds__(kRowsWarps * 32, 1) decode_step_rows_kernel(const __grid_constant__ StepParams p) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // Programmatic stream serialization as in decode_step_kernel: only the set-up of shared memory
    // runs ahead of the preceding kernel's completion.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    constexpr uint32_t kBarsAll = kRowsWarps * kRowsRing;
    constexpr uint32_t kZeroRow = kBarsAll + kRowsWarps * kRowsSlots * (uint32_t)sizeof(uint64_t);
    constexpr uint32_t kDescsAll = kZeroRow + 128;
    if (threadIdx.x < 32) *sp<uint32_t>(kZeroRow + threadIdx.x * 4) = 0u;
    if (lane == 0) {
        for (int s = 0; s < kRowsSlots; ++s) mbar_init(sp<uint64_t>(kBarsAll + ((uint32_t)warp * kRowsSlots + s) * 8), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    __shared__ unsigned aan_next;
    if (threadIdx.x == 0) aan_next = 0u;
    if (p.n_items == 0) { __syncthreads(); aan_chunks<__nv_bfloat16>(p, lane, &aan_next); return; }

    __shared__ unsigned q_next, warp_count[kRowsWarps];
    ItemDesc* descs = sp<ItemDesc>(kDescsAll);

    RowWarp w(p);
    w.sm_base = smem_u32(san_smem);
    w.ring = (uint32_t)warp * kRowsRing;
    w.bars = kBarsAll + (uint32_t)warp * kRowsSlots * 8;
    w.descs_off = kDescsAll; w.q_next = &q_next; w.zero_row = w.sm_base + kZeroRow;
    w.lane = lane;
    w.head_v = w.tail_v = w.head_p = 0; w.n_slots = w.n_ret = 0; w.rec_base = w.rec_end = w.rec_grp = 0; w.n_groups = 0;
    w.dead = false; w.p_active = false; w.p_plane = 0; w.p_idx = 0;

    const unsigned long long my_slots = (p.n_items > blockIdx.x) ? ((unsigned long long)p.n_items - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    if (my_slots == 0) { __syncthreads(); aan_chunks<__nv_bfloat16>(p, lane, &aan_next); }
    for (unsigned long long k0 = 0; k0 < my_slots; k0 += kCtaItems) {
        // -- decode: thread t takes slot k0 + t; survivors keep their order (big items first)
        ItemDesc mine;
        bool ok = false;
        if (threadIdx.x < kCtaItems && k0 + threadIdx.x < my_slots)
            ok = decode_item<128>(p, (unsigned)((k0 + threadIdx.x) * gridDim.x + blockIdx.x), &mine);
        const unsigned ballot = __ballot_sync(0xffffffffu, ok);
        if (lane == 0) warp_count[warp] = __popc(ballot);
        __syncthreads();                                 // also: every warp is done with the previous round's items
        if (threadIdx.x == 0) q_next = kRowsWarps;       // the first kRowsWarps items go to the warps directly
        static_assert(kRowsWarps <= 32, "one lane per warp");
        const unsigned cnt = lane < kRowsWarps ? warp_count[lane] : 0u;
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
        // One plane per turn: the item in hand is `c_idx`, its next plane `c_plane` (0 = keys, l + 1 = the
        // values of its layer l).  More planes are requested when an item starts (what the item before
        // gave back goes to the items behind this one) and while a fat item's own planes are not all out.
        uint32_t pw[2 * kRowsMaxBlocks];
        unsigned c_idx = 0;
        int c_plane = 0;
        bool have = false;
        while (!w.dead) {
            if (!have || (w.p_active && w.p_idx == c_idx)) w.top_up();
            if (!have) {
                if (w.fifo_n == 0) break;
                c_idx = (unsigned)(w.fifo & 0xffull);
                w.fifo >>= 8; w.fifo_n -= 1;
                c_plane = 0; have = true;
            }
            const ItemDesc& d = w.desc(c_idx);
            const uint32_t st = w.acquire();
            if (st == RowWarp::kNoPlane) break;
            const int nb = (d.n + 15) >> 4;
            if (c_plane == 0) {
                if (nb <= 2) w.scores<2>(d, st, pw); else if (nb <= 4) w.scores<4>(d, st, pw); else w.scores<6>(d, st, pw);
            } else {
                if (nb <= 2) w.apply<2>(d, st, pw, c_plane - 1); else if (nb <= 4) w.apply<4>(d, st, pw, c_plane - 1); else w.apply<6>(d, st, pw, c_plane - 1);
            }
            w.release();
            if (c_plane == d.pi) have = false; else c_plane += 1;
        }
        if (k0 == 0) aan_chunks<__nv_bfloat16>(p, lane, &aan_next);
    }
}

}  // namespace san
