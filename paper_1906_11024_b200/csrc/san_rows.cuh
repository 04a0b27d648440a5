// One decode step in one launch for sentence-sized rows (every row at most kRowsMaxPos
// positions, bf16): cache append, weights (Eq. 1) and apply (Eq. 2 with Eq. 4) for every block
// of both attention kinds, plus the AAN running average.
//
// The list of work items, their decoding and their hand-out to the warps of a CTA are those of
// decode_step_kernel.  What differs is how a warp works through an item, because with rows this
// short a step is as long as the chain of dependent instructions and memory round trips of the
// items one warp takes one after the other:
//   * an item is R heads (1, 2 or 4) of one (block, sequence), so that what an item costs beside
//     its arithmetic is paid once for all of them and their independent chains overlap;
//   * a whole plane of an item (its key rows, or the value rows of one layer, of all its heads) is
//     one slot of the warp's ring, which holds planes of any size back to back, and the planes of
//     the next items are requested while the warp still computes on this one.  The warp fetches
//     them itself in 16-byte pieces (cp.async, one group per plane): a bulk copy costs its warp
//     some 400 cycles to issue however small it is, and more when all warps of an SM issue at once
//     (measured: a third of a warp's time went into issuing them), while a plane of 20 rows is five
//     cp.async instructions.  This step's own key / value row (not yet in the cache) and the query
//     rows come the same way, the former already chunk-permuted like a cached row, so that the
//     arithmetic sees one uniform tile;
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

constexpr int kRowsWarps = 12;
constexpr int kRowsRing = 17792;        // bytes per warp: 139 rows
constexpr int kRowsRingRows = kRowsRing / 128;
constexpr int kRowsSlots = 8;           // planes in flight per warp at most (one cp.async group each)
constexpr int kRowsMaxBlocks = 6;
constexpr int kRowsMaxPos = 16 * kRowsMaxBlocks;   // positions per row at most
constexpr int kRowsMaxWeights = 24;     // bf16 pairs of weights an item keeps in registers: heads x 2 x blocks

enum { TAG_ROWS = 9 };

// Blocks of 16 positions an item of `heads` heads may have (its weights stay in registers).
__host__ __device__ constexpr int rows_max_blocks(int heads) { return heads == 4 ? 3 : heads == 2 ? 5 : kRowsMaxBlocks; }

constexpr size_t rows_smem_bytes() {
    return (size_t)kRowsWarps * kRowsRing + 128 /* a row of zeros */ + (size_t)kCtaItems * sizeof(ItemDesc);
}

// D(16x8) += A(16x16) * B(16x8) where rows 8..15 of A are zero.  d[2], d[3] (rows 8..15 of D) stay
// zero; they are carried along because the instruction takes its accumulator as four registers in a row.
__device__ __forceinline__ void mma_bf16_top(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%5}, {%7,%8}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(0u), "r"(a2), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ float ex2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct RowWarp {
    const StepParams& p;
    uint32_t sm_base;             // shared-space address of san_smem
    uint32_t ring;                // offset of this warp's ring
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
    uint32_t rec_base, rec_end;   // lane i < kRowsSlots: offset of the plane with sequence number i (mod kRowsSlots), head_v behind it
    unsigned long long fifo;      // items whose planes are (being) requested and whose arithmetic is still to do
    int fifo_n;
    bool dead;                    // the ring's bookkeeping broke (reported as an error): leave

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

    // Requests, in order, as many of the planes still to come as the ring has room for (at most
    // kRowsSlots at a time).  A plane of an item with R heads is R runs of cached rows (the heads'
    // panels lie apart in the cache and side by side in the slot), this step's own row of every head
    // where it closes the plane, and, behind the key plane, the query rows.  One cp.async group each.
    __device__ __forceinline__ void top_up() {
        while (p_active && n_slots - n_ret < (uint32_t)kRowsSlots) {
            const ItemDesc& d = desc(p_idx);
            const int n = d.n, has_new = d.has_new, R = d.heads, pi = d.pi;
            const int nqr = p_plane == 0 ? R * d.nq : 0;               // the query rows ride behind the key rows
            const uint32_t bytes = (uint32_t)(R * n + nqr) * 128u;
            uint32_t hv = head_v, hp = head_p;
            if (hp + bytes > (uint32_t)kRowsRing) { hv += (uint32_t)kRowsRing - hp; hp = 0; }     // a plane is contiguous
            if (hv + bytes - tail_v > (uint32_t)kRowsRing) break;
            const uint32_t base = ring + hp;
            head_v = hv + bytes; head_p = hp + bytes;
            if ((uint32_t)lane == n_slots % kRowsSlots) { rec_base = base; rec_end = head_v; }
            const KindParams& kp = p.k[d.kind];
            const char* src = p_plane == 0 ? d.srcK : d.srcV + (long long)(p_plane - 1) * kp.plane_bytes;
            const uint32_t dst = sm_base + base + (uint32_t)lane * 16u;
            const int cached = (n - has_new) * 8;                        // 16-byte pieces of a head's cached rows
            src += lane * 16;
            for (int hh = 0; hh < R; ++hh) {
                const char* sh = src + (unsigned long long)hh * kp.panel_bytes;
                const uint32_t dh = dst + (uint32_t)(hh * n) * 128u;
#pragma unroll 4
                for (int i = 0; i < cached; i += 32)
                    if (i + lane < cached) cp_async_16(dh + i * 16, sh + i * 16);
            }
            if (has_new) {      // this step's row of every head, chunk-permuted like a cached row: piece (head, chunk) per lane
                const char* nw = p_plane == 0 ? d.knew : d.vnew + (long long)(p_plane - 1) * kp.layer_bytes;
                const int hh = lane >> 3, c = lane & 7;
                if (hh < R) cp_async_16(sm_base + base + (uint32_t)(hh * n + n - 1) * 128u + (uint32_t)((c ^ ((n - 1) & 7)) << 4), nw + hh * 128 + c * 16);
            }
            if (nqr) {          // query row hh * nq + qi: chunk c at c ^ (row & 7)
                const int nq = d.nq;
                const unsigned q_stride = (unsigned)p.H * 128u;
                for (int i = lane; i < nqr * 8; i += 32) {
                    const int r = i >> 3, c = i & 7;
                    int hh = 0;
                    if (r >= nq) hh = 1;
                    if (r >= 2 * nq) hh = 2;
                    if (r >= 3 * nq) hh = 3;
                    cp_async_16(sm_base + base + (uint32_t)(R * n + r) * 128u + (uint32_t)((c ^ (r & 7)) << 4),
                                d.q + hh * 128 + (unsigned long long)(r - hh * nq) * q_stride + c * 16);
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            n_slots += 1;
            if (p_plane == pi) next_item(); else p_plane += 1;
        }
    }

    // Waits for the next plane in order; returns the offset of its rows, or kNoPlane if it was never requested.
    static constexpr uint32_t kNoPlane = 0xffffffffu;
    __device__ __forceinline__ uint32_t acquire() {
        if (n_ret == n_slots) { fail(100); return kNoPlane; }      // top_up always finds room in an empty ring
        // groups complete in order: all but the planes requested after this one
        switch (n_slots - n_ret - 1u) {
            case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
            case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
            case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
            case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
            case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
            case 5: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
            case 6: asm volatile("cp.async.wait_group 6;" ::: "memory"); break;
            default: asm volatile("cp.async.wait_group 7;" ::: "memory"); break;
        }
        __syncwarp();
        return __shfl_sync(0xffffffffu, rec_base, (int)(n_ret % kRowsSlots));
    }
    // Every lane is done with the plane: its bytes are free again.
    __device__ __forceinline__ void release() {
        __syncwarp();
        tail_v = __shfl_sync(0xffffffffu, rec_end, (int)(n_ret % kRowsSlots));
        n_ret += 1;
        if (n_ret == n_slots) { tail_v = head_v; head_p = 0; }      // nothing outstanding: the next plane starts the ring afresh
    }

    template <int NB, int NBLO, int R> __device__ __forceinline__ void scores(const ItemDesc& d, uint32_t st, uint32_t (&pw)[kRowsMaxWeights]);
    template <int NB, int NBLO, int R> __device__ __forceinline__ void apply(const ItemDesc& d, uint32_t st, const uint32_t (&pw)[kRowsMaxWeights], int l);
};

// The key plane of an item of R heads with more than NBLO and at most NB blocks of 16 positions (at
// st: the heads' key rows one head after the other, then their query rows): this step's key row to
// the cache, scores, softmax in registers, S to the caller; leaves the weights as bf16 pairs in pw
// (head hh at pw[hh * 2 NB ..]), the A fragments of the apply products.  Cached rows keep chunk c
// at c ^ (position & 7), and so does this step's own row in the slot; query row r keeps chunk c at c ^ (r & 7).
template <int NB, int NBLO, int R>
__device__ __forceinline__ void RowWarp::scores(const ItemDesc& d, uint32_t st, uint32_t (&pw)[kRowsMaxWeights]) {
    static_assert(R * 2 * NB <= kRowsMaxWeights, "the weights of all heads stay in registers");
    const int n = d.n, nq = d.nq, has_new = d.has_new;
    const int tig = lane & 3, gid = lane >> 2;                 // mma fragment coordinates
    const int r8 = lane & 7, m4 = lane >> 3;                   // ldmatrix: this lane addresses row r8 of matrix m4
    const uint32_t st_s = sm_base + st;
    const KindParams& kp = p.k[d.kind];
    const float scl = p.scale_log2e;
    const int lim = n - 2 * tig;                               // position 8 j + 2 tig + e is in the row iff 8 j + e < lim
#pragma unroll
    for (int hh = 0; hh < R; ++hh) {
        if (has_new && d.lead && lane < 8)                      // this step's key row into the cache (already permuted)
            *reinterpret_cast<uint4*>(const_cast<char*>(d.srcK) + (unsigned long long)hh * kp.panel_bytes + (n - 1) * 128 + lane * 16) =
                *sp<uint4>(st + (uint32_t)(hh * n + n - 1) * 128u + lane * 16);
        // A fragments of the queries: matrix m4 = rows 0..7, 16-byte chunk 4 kp + m4; registers (a0, a2) of
        // k-steps 2 kp and 2 kp + 1.  Rows 8..15 are zero and never loaded; rows at or beyond nq read zeros.
        uint32_t qa[4][2];
        {
            const uint32_t qr = (uint32_t)(hh * nq + r8);
            const uint32_t a = (r8 < nq) ? st_s + ((uint32_t)(R * n) + qr) * 128u + (((uint32_t)m4 ^ (qr & 7u)) << 4) : zero_row;
            const uint32_t flip = (r8 < nq) ? 64u : 0u;
            uint32_t r[4];
            ldsm_x4(a, r);        qa[0][0] = r[0]; qa[0][1] = r[1]; qa[1][0] = r[2]; qa[1][1] = r[3];
            ldsm_x4(a ^ flip, r); qa[2][0] = r[0]; qa[2][1] = r[1]; qa[3][0] = r[2]; qa[3][1] = r[3];
        }
        // B fragments of 8 positions: matrix m4 = positions 8 j + r8, chunk 4 kp + m4; registers (b0, b1)
        // of k-steps 2 kp and 2 kp + 1.
        float sc[2 * NB][2];
        const uint32_t ka = st_s + (uint32_t)(hh * n + r8) * 128u + (uint32_t)((m4 ^ r8) << 4);
#pragma unroll
        for (int j = 0; j < 2 * NB; ++j) {
            const uint32_t kj = ka + j * 1024;
            uint32_t b0[4], b1[4];
            ldsm_x4(kj, b0);
            ldsm_x4(kj ^ 64u, b1);
            float c[4] = {0.f, 0.f, 0.f, 0.f};
            mma_bf16_top(c, qa[0][0], qa[0][1], b0[0], b0[1]);
            mma_bf16_top(c, qa[1][0], qa[1][1], b0[2], b0[3]);
            mma_bf16_top(c, qa[2][0], qa[2][1], b1[0], b1[1]);
            mma_bf16_top(c, qa[3][0], qa[3][1], b1[2], b1[3]);
            sc[j][0] = c[0]; sc[j][1] = c[1];
        }
        // Softmax in registers: sc[j][e] is query gid, position 8 j + 2 tig + e (log2 domain after scaling).
        // Positions at or beyond n (the next head's rows, the query rows, stale bytes) are masked out.
        float mx = -INFINITY;
#pragma unroll
        for (int j = 0; j < 2 * NB; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const float v = (j < 2 * NBLO || 8 * j + e < lim) ? sc[j][e] * scl : -INFINITY;
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
        float* Srow = (d.S && gid < nq) ? d.S + (long long)hh * kp.S_ld + (long long)gid * ((long long)p.H * kp.S_ld) + 2 * tig : nullptr;
#pragma unroll
        for (int j = 0; j < 2 * NB; ++j) {
            const float w0 = sc[j][0] * inv, w1 = sc[j][1] * inv;
            if (Srow) {
                if (j < 2 * NBLO || 8 * j < lim) Srow[8 * j] = w0;
                if (j < 2 * NBLO || 8 * j + 1 < lim) Srow[8 * j + 1] = w1;
            }
            pw[hh * 2 * NB + j] = pack_bf16x2(w0, w1);
        }
    }
}

// The value plane of the item's layer l (at st): this step's value row to the cache, S . V, output.
// B fragments through ldmatrix.trans: matrix m4 = positions 16 kk + 8 (m4 & 1) + r8, chunk
// 2 jp + (m4 >> 1); registers (b0, b1) of dim tiles 2 jp and 2 jp + 1.  Rows at or beyond n hold other
// bytes: their weights are zero, but 0 x NaN would not be, so those lanes address a row of zeros.
template <int NB, int NBLO, int R>
__device__ __forceinline__ void RowWarp::apply(const ItemDesc& d, uint32_t st, const uint32_t (&pw)[kRowsMaxWeights], int l) {
    const int n = d.n, has_new = d.has_new;
    const int tig = lane & 3, gid = lane >> 2;
    const int r8 = lane & 7, m4 = lane >> 3;
    const KindParams& kp = p.k[d.kind];
    const uint32_t st_s = sm_base + st;
    const int vpos = 8 * (m4 & 1) + r8;
    const bool writes = gid < d.nq;
    char* op = d.O + (long long)l * kp.layer_bytes + (long long)gid * ((long long)p.H * 128) + tig * 4;
    char* vdst = const_cast<char*>(d.srcV) + (long long)l * kp.plane_bytes + (n - 1) * 128 + lane * 16;
#pragma unroll
    for (int hh = 0; hh < R; ++hh) {
        if (has_new && lane < 8)
            *reinterpret_cast<uint4*>(vdst + (unsigned long long)hh * kp.panel_bytes) = *sp<uint4>(st + (uint32_t)(hh * n + n - 1) * 128u + lane * 16);
        const uint32_t va = st_s + (uint32_t)(hh * n + vpos) * 128u + (uint32_t)(((m4 >> 1) ^ r8) << 4);
        float acc[8][4];
#pragma unroll
        for (int x = 0; x < 8; ++x) { acc[x][0] = 0.f; acc[x][1] = 0.f; acc[x][2] = 0.f; acc[x][3] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < NB; ++kk) {
            const uint32_t vk = va + kk * 2048;
            const bool in_row = kk < NBLO || 16 * kk + vpos < n;
            uint32_t b[4][4];
#pragma unroll
            for (int jp = 0; jp < 4; ++jp) ldsm_x4_t(in_row ? vk ^ (uint32_t)(jp << 5) : zero_row, b[jp]);
#pragma unroll
            for (int jp = 0; jp < 4; ++jp) {
                mma_bf16_top(acc[2 * jp], pw[hh * 2 * NB + 2 * kk], pw[hh * 2 * NB + 2 * kk + 1], b[jp][0], b[jp][1]);
                mma_bf16_top(acc[2 * jp + 1], pw[hh * 2 * NB + 2 * kk], pw[hh * 2 * NB + 2 * kk + 1], b[jp][2], b[jp][3]);
            }
        }
        // acc[x][0], [1]: query gid, dims 8 x + 2 tig, + 1
        if (writes) {
#pragma unroll
            for (int x = 0; x < 8; ++x) *reinterpret_cast<uint32_t*>(op + hh * 128 + x * 16) = pack_bf16x2(acc[x][0], acc[x][1]);
        }
    }
}

__global__ void __launch_bounds__(kRowsWarps * 32, 1) decode_step_rows_kernel(const __grid_constant__ StepParams p) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // Programmatic stream serialization as in decode_step_kernel: only the set-up of shared memory
    // runs ahead of the preceding kernel's completion.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    constexpr uint32_t kZeroRow = kRowsWarps * kRowsRing;
    constexpr uint32_t kDescsAll = kZeroRow + 128;
    if (threadIdx.x < 32) *sp<uint32_t>(kZeroRow + threadIdx.x * 4) = 0u;
    asm volatile("griddepcontrol.wait;" ::: "memory");

    __shared__ unsigned aan_next;
    if (threadIdx.x == 0) aan_next = 0u;
    if (p.n_items == 0) { __syncthreads(); aan_chunks<__nv_bfloat16>(p, lane, &aan_next); return; }

    __shared__ unsigned q_next, warp_count[kRowsWarps];
    ItemDesc* descs = sp<ItemDesc>(kDescsAll);

    RowWarp w(p);
    w.sm_base = smem_u32(san_smem);
    w.ring = (uint32_t)warp * kRowsRing;
    w.descs_off = kDescsAll; w.q_next = &q_next; w.zero_row = w.sm_base + kZeroRow;
    w.lane = lane;
    w.head_v = w.tail_v = w.head_p = 0; w.n_slots = w.n_ret = 0; w.rec_base = w.rec_end = 0;
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
        uint32_t pw[kRowsMaxWeights];
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
            const int nb = (d.n + 15) >> 4, R = d.heads, l = c_plane - 1;
#define SAN_ROWS_PLANE(NB, NBLO, RR) do { if (c_plane == 0) w.scores<NB, NBLO, RR>(d, st, pw); else w.apply<NB, NBLO, RR>(d, st, pw, l); } while (0)
            if (R == 1) {
                if (nb <= 2) SAN_ROWS_PLANE(2, 0, 1); else if (nb <= 4) SAN_ROWS_PLANE(4, 2, 1); else SAN_ROWS_PLANE(6, 4, 1);
            } else if (R == 2) {
                if (nb <= 2) SAN_ROWS_PLANE(2, 0, 2); else if (nb == 3) SAN_ROWS_PLANE(3, 2, 2); else if (nb == 4) SAN_ROWS_PLANE(4, 3, 2); else SAN_ROWS_PLANE(5, 4, 2);
            } else {
                if (nb <= 2) SAN_ROWS_PLANE(2, 0, 4); else SAN_ROWS_PLANE(3, 2, 4);
            }
#undef SAN_ROWS_PLANE
            w.release();
            if (c_plane == d.pi) have = false; else c_plane += 1;
        }
        if (k0 == 0) aan_chunks<__nv_bfloat16>(p, lane, &aan_next);
    }
}

}  // namespace san
