// Full-sequence shared attention on the fifth-generation tensor cores (tcgen05, accumulators
// in tensor memory), for sequences long enough to fill a 128-query tile.  Same operation as
// full_block_kernel: S = Softmax(Q.K^T / 8) once per block (Eq. 1, Eq. 3), O_l = S.V_l for each
// layer of the block (Eq. 2, Eq. 4).
//
// CTA = (128 queries, head, sequence), kTcThreads threads; query row r is lane r of tensor
// memory and belongs to threads r, r + 128, ..., which share a chunk's 64 score columns (a warp
// reaches the 32 lanes of its rank modulo 4).  Row statistics are thread-local and joined once,
// through shared memory, between the passes (no shuffles).  A run is 2 x chunks steps:
//   pass 0  per chunk of 64 keys one tcgen05.mma chain (M 128, N 64, K 64) writes the scores
//           into tensor memory; each thread reads its part of its row back and keeps a running
//           (max, sum).
//   pass 1  scores once more (cheaper than keeping 128 x l floats); weights =
//           exp2(z - max) / sum go out to S and, as a bf16 high part and a bf16 remainder, into
//           two shared-memory operand tiles; two MMA chains per group of up to four layers
//           (N = 64 x layers) add weights x values to the layers' accumulators, which stay in
//           tensor memory (columns 64 + 64 l) until the last chunk.
// The tensor pipe runs ahead of the threads: the scores of step t + 1 go to a second score
// buffer while the threads work on step t, and the outputs of step t - 1 are still being
// accumulated; key chunks are copied (cp.async) three steps ahead, value chunks one.
// Operand tiles are rows of 128 bytes with the 16-byte chunks XOR-swizzled by (row & 7), the
// 128-byte swizzle the matrix descriptors name; queries, keys and weights are K-major, the
// value rows (dims contiguous) are the MN-major B operand.  Every wait on the MMA barrier is
// bounded; a CTA whose wait runs out stops issuing, frees its tensor memory and leaves its
// outputs unwritten.
#pragma once

#include "san_full.cuh"
#include "san_fused.cuh"

namespace san {

constexpr int kTcQ = 128;                 // queries per CTA = tensor-memory lanes
constexpr int kTcChunk = 64;              // keys per MMA chain
constexpr int kTcThreads = 256;
constexpr int kTcSplit = kTcThreads / kTcQ;   // threads per query row; each takes 64 / kTcSplit score columns
constexpr int kTcCols1 = kTcChunk / kTcSplit;  // score columns per thread
// Apply the weights as a bf16 high part plus a bf16 remainder (two MMAs per key step) or as the high
// part alone.  The outputs are bf16: their own rounding (2^-9) is what shows against the float64
// reference either way (tolerance 1e-2), so the remainder is left out.
constexpr bool kTcRemainder = false;
constexpr int kTcMaxLayers = 6;           // accumulators: 64 columns each after the 64 of the scores (512 columns in all)
constexpr int kTcCols = 512;
constexpr uint32_t kTcScores1 = 448;       // second score buffer: the 64 columns behind the six accumulators
constexpr uint32_t kTcTileQ = kTcQ * 128, kTcTileK = kTcChunk * 128;      // bytes of a 128-row and of a 64-row operand tile

// shared-memory matrix descriptor: 128-byte swizzle, 8-row groups 1024 bytes apart; lead_bytes =
// distance between the 64-element column blocks of an MN-major operand wider than 64 (else unused)
__device__ __forceinline__ uint64_t tc_desc(uint32_t smem_addr, uint32_t lead_bytes = 16) {
    return (uint64_t)((smem_addr >> 4) & 0x3fffu) | ((uint64_t)((lead_bytes >> 4) & 0x3fffu) << 16) |
           ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// instruction descriptor: float32 accumulator, bf16 operands, M 128, N n; b_mn: B is MN-major
__device__ __forceinline__ uint32_t tc_idesc(bool b_mn, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn ? (1u << 16) : 0u) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
    const uint32_t none = 0u;      // no output lane is disabled
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n}"
                 :: "r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(accumulate), "r"(none) : "memory");
}
// 2^x in one instruction (relative error about 2^-22, far inside the tolerance of S; 2^-inf = 0)
__device__ __forceinline__ float tc_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void tc_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void tc_ld(uint32_t taddr, float (&v)[16]) { tc_ld16(taddr, v); }
__device__ __forceinline__ void tc_ld(uint32_t taddr, float (&v)[32]) { tc_ld32(taddr, v); }

// rows [0, rows) of a [n][64] bf16 panel (row stride row_elems) into a swizzled 64-row operand
// tile with 16-byte asynchronous copies (no registers held while they fly); the other rows are
// zero-filled (a copy of source size 0).  Consecutive threads take consecutive pieces.
__device__ __forceinline__ void tc_stage_async(uint32_t tile_s, const __nv_bfloat16* src, long long row_elems, int rows) {
#pragma unroll
    for (int i = 0; i < kTcChunk * 8 / kTcThreads; ++i) {
        const int u = (int)threadIdx.x + i * kTcThreads, r = u >> 3, c = u & 7;
        const uint32_t bytes = r < rows ? 16u : 0u;
        const __nv_bfloat16* from = src + (long long)(r < rows ? r : 0) * row_elems + c * 8;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;"
                     :: "r"(tile_s + (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4))), "l"(from), "r"(bytes) : "memory");
    }
}

extern __shared__ __align__(1024) unsigned char tc_smem[];

static __global__ void __launch_bounds__(kTcThreads, 1) full_block_tc5_kernel(const FullParams p) {
    const int seq = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * kTcQ;
    const int len = min(p.lens[seq], p.max_len);
    if (q0 >= len) return;                                   // uniform over the CTA, before anything is allocated
    const int row = threadIdx.x & (kTcQ - 1), part = threadIdx.x >> 7, warp = threadIdx.x >> 5;
    const int qrow = q0 + row;
    const long long row_elems = (long long)p.H * kDh;
    const long long seq_off = ((long long)seq * p.cap) * row_elems + (long long)h * kDh;
    const int n_keys = p.causal ? min(len, q0 + kTcQ) : len;
    const int n_chunks = (n_keys + kTcChunk - 1) / kTcChunk;

    // shared memory (1024-byte aligned tiles): Q | weights high | weights remainder | a ring of four
    // K chunks | a ring of two (V chunk of each layer).  Keys are needed a step before the values of
    // the same chunk (the scores run ahead), so they are copied three steps ahead, values one.
    unsigned char* base = tc_smem + ((1024u - (smem_u32(tc_smem) & 1023u)) & 1023u);
    unsigned char* sQ = base;
    unsigned char* sPh = sQ + kTcTileQ;
    unsigned char* sPl = sPh + kTcTileQ;
    const uint32_t sKr = smem_u32(sPl + kTcTileQ);                     // K chunk of step t at sKr + (t % 4) * kTcTileK
    const uint32_t sVr = sKr + 4 * kTcTileK;                            // V chunks of step t at sVr + (t % 2) * kVBuf, layer l at + l * kTcTileK
    const uint32_t kVBuf = (uint32_t)p.n_layers * kTcTileK;
    __shared__ __align__(8) uint64_t bar[2];         // completion of the score MMAs / of the output MMAs
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead_s;
    __shared__ float2 stats_s[kTcSplit][kTcQ];       // (max, sum) of each part of a row after pass 0

    if (threadIdx.x == 0) {
        mbar_init(&bar[0], 1);
        mbar_init(&bar[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        dead_s = 0;
    }
    __syncwarp();
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&tmem_base_s)), "r"((uint32_t)kTcCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // this thread's query row into the Q tile (zero beyond the sequence)
    {
        const __nv_bfloat16* qsrc = p.q + seq_off + (long long)qrow * row_elems;
#pragma unroll
        for (int c = part * (8 / kTcSplit); c < (part + 1) * (8 / kTcSplit); ++c) {
            const uint4 val = qrow < len ? ld16_stream(qsrc + c * 8) : make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4*>(sQ + row * 128 + ((c ^ (row & 7)) << 4)) = val;
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_base_s;
    const uint32_t t_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(part * kTcCols1);   // this warp's 32 lanes, this thread's columns of every 64
    const uint32_t bar_s = smem_u32(&bar[0]), bar_o = smem_u32(&bar[1]);
    const uint64_t dQ = tc_desc(smem_u32(sQ)), dPh = tc_desc(smem_u32(sPh)), dPl = tc_desc(smem_u32(sPl));
    const uint32_t idS = tc_idesc(false, kTcChunk);
    uint32_t phase_s = 0, phase_o = 0;
    bool dead = false;
    const int n_steps = 2 * n_chunks;             // step t: pass t / n_chunks, chunk t % n_chunks

    // Bounded wait on one of the two MMA barriers; a wait that runs out marks the CTA dead (seen by
    // everyone after the next CTA barrier).
    auto mma_wait = [&](uint32_t bar_addr, uint32_t& phase) {
        if (!mbar_try_wait(bar_addr, phase) && !mbar_wait_slow(bar_addr, phase)) dead_s = 1;
        phase ^= 1u;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    };
    // Copies of step t, each a group of its own (empty where the step has none): the key chunk, and in
    // pass 1 the value chunk of every layer.
    auto issue_keys = [&](int t) {
        if (t < n_steps) {
            const int k0 = (t >= n_chunks ? t - n_chunks : t) * kTcChunk;
            tc_stage_async(sKr + (uint32_t)(t & 3) * kTcTileK, p.k + seq_off + (long long)k0 * row_elems, row_elems, min(kTcChunk, len - k0));
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    auto issue_values = [&](int t) {
        if (t >= n_chunks && t < n_steps) {
            const int k0 = (t - n_chunks) * kTcChunk, rows = min(kTcChunk, len - k0);
            for (int l = 0; l < p.n_layers; ++l)
                tc_stage_async(sVr + (uint32_t)(t & 1) * kVBuf + (uint32_t)l * kTcTileK,
                               p.v + (long long)l * p.layer_elems + seq_off + (long long)k0 * row_elems, row_elems, rows);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // Scores of step t: Q x (key chunk t)^T into score buffer t & 1 of tensor memory.
    auto issue_scores = [&](int t) {
        const uint64_t dK = tc_desc(sKr + (uint32_t)(t & 3) * kTcTileK);
        const uint32_t d = tmem + ((t & 1) ? kTcScores1 : 0u);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)            // 16 dims = 32 bytes along a row per step
            tc_mma(d, dQ + 2 * ks, dK + 2 * ks, idS, ks > 0 ? 1u : 0u);
        tc_commit(bar_s);
    };

    // The tensor pipe runs ahead of the threads: when the threads turn the scores of step t into
    // statistics or weights, the scores of step t + 1 are being computed (second score buffer) and,
    // in pass 1, so are the outputs of step t - 1.  Every step commits two copy groups, keys of
    // step t + 3 and values of step t + 1; the set-up commits what steps -3 .. -1 would have.
    issue_keys(0); issue_values(-2);
    issue_keys(1); issue_values(-1);
    issue_keys(2); issue_values(0);
    asm volatile("cp.async.wait_group 5;" ::: "memory");             // keys of step 0 have landed
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        issue_scores(0);
    }
    float m_run = -INFINITY, s_run = 0.f, inv = 0.f;
    for (int t = 0; t < n_steps; ++t) {
        const int pass = t >= n_chunks ? 1 : 0, kc = t - pass * n_chunks, k0 = kc * kTcChunk;
        mma_wait(bar_s, phase_s);                 // scores of step t (and everything issued before them) are complete
        float z[kTcCols1];                        // this thread's part of the row's 64 scores
        tc_ld(t_lane + ((t & 1) ? kTcScores1 : 0u), z);
        asm volatile("cp.async.wait_group 3;" ::: "memory");         // keys of step t + 1 have landed (this thread's copies)
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();                          // ... everyone's; and everyone has read the scores of step t
        if (dead_s) { dead = true; break; }
        if (threadIdx.x == 0 && t + 1 < n_steps) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            issue_scores(t + 1);
        }
        issue_keys(t + 3);                        // into the slot of step t - 1, whose scores are complete
        if (pass == 0) issue_values(t + 1);       // (a real copy only ahead of the first step of pass 1)
        if (t == n_chunks) {                      // between the passes: join the two halves of every row
            stats_s[part][row] = make_float2(m_run, s_run);
            __syncthreads();
            float m_all = -INFINITY, s_all = 0.f;
#pragma unroll
            for (int o = 0; o < kTcSplit; ++o) m_all = fmaxf(m_all, stats_s[o][row].x);
            if (m_all > -INFINITY) {
#pragma unroll
                for (int o = 0; o < kTcSplit; ++o) s_all += stats_s[o][row].y * exp2f(stats_s[o][row].x - m_all);
            }
            m_run = m_all; s_run = s_all;
            inv = s_run > 0.f ? 1.0f / s_run : 0.f;
        }
        const int kh = k0 + part * kTcCols1;      // first key of this thread's part
        float m_chunk = -INFINITY;
        // z stays unscaled: the scale (positive, so it commutes with the maximum) is folded into the
        // exponent's argument, ex2(z * scale - m), one multiply-add per score
        const float sc = p.scale_log2e;
        if (k0 + kTcChunk <= len && (!p.causal || k0 + kTcChunk - 1 <= q0)) {
            // every row of the tile sees every key of the chunk (uniform over the CTA): no masks
#pragma unroll
            for (int j = 0; j < kTcCols1; ++j) m_chunk = fmaxf(m_chunk, z[j]);
        } else {
#pragma unroll
            for (int j = 0; j < kTcCols1; ++j) {
                const int key = kh + j;
                const bool ok = key < len && (!p.causal || key <= qrow);
                z[j] = ok ? z[j] : -INFINITY;
                m_chunk = fmaxf(m_chunk, z[j]);
            }
        }
        m_chunk *= sc;
        if (pass == 0) {
            const float m_new = fmaxf(m_run, m_chunk);
            if (m_new > -INFINITY) {
                float s = s_run * exp2f(m_run - m_new);
#pragma unroll
                for (int j = 0; j < kTcCols1; ++j) s += tc_ex2(fmaf(z[j], sc, -m_new));
                s_run = s; m_run = m_new;
            }
            continue;
        }
        // ---- pass 1: weights of this chunk, in registers first
        float* Srow = (p.S && qrow < len) ? p.S + (((long long)seq * p.H + h) * p.cap + qrow) * p.ld_s + kh : nullptr;
        const float m_use = m_run > -INFINITY ? m_run : 0.f;
        uint32_t hi[kTcCols1 / 2], lo[kTcCols1 / 2];
#pragma unroll
        for (int e = 0; e < kTcCols1 / 2; ++e) {
            const float w0 = tc_ex2(fmaf(z[2 * e], sc, -m_use)) * inv, w1 = tc_ex2(fmaf(z[2 * e + 1], sc, -m_use)) * inv;
            z[2 * e] = w0; z[2 * e + 1] = w1;
            hi[e] = full_pack(w0, w1);
            if (kTcRemainder) lo[e] = full_pack(w0 - __uint_as_float(hi[e] << 16), w1 - __uint_as_float(hi[e] & 0xffff0000u));
        }
        if (Srow) {
#pragma unroll
            for (int j = 0; j < kTcCols1; ++j)
                if (kh + j < len) Srow[j] = z[j];                  // keys a causal row does not see are stored as 0
        }
        if (kc > 0) mma_wait(bar_o, phase_o);     // outputs of step t - 1 complete: the weight tiles and its buffer are free
        issue_values(t + 1);                      // into the slot of step t - 1
#pragma unroll
        for (int c = 0; c < kTcCols1 / 8; ++c) {  // 8 keys = one 16-byte chunk of the operand rows; this part owns chunks part * kTcCols1 / 8 ..
            const int at = row * 128 + (((part * (kTcCols1 / 8) + c) ^ (row & 7)) << 4);
            *reinterpret_cast<uint4*>(sPh + at) = make_uint4(hi[4 * c], hi[4 * c + 1], hi[4 * c + 2], hi[4 * c + 3]);
            if (kTcRemainder) *reinterpret_cast<uint4*>(sPl + at) = make_uint4(lo[4 * c], lo[4 * c + 1], lo[4 * c + 2], lo[4 * c + 3]);
        }
        asm volatile("cp.async.wait_group 2;" ::: "memory");         // values of step t have landed
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (dead_s) { dead = true; break; }
        if (threadIdx.x == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            // Up to four layers per MMA: their value tiles lie one behind the other (8 KB apart) and
            // form one MN-major B operand of 64 dims x layers columns; so do their accumulators.
            for (int l0 = 0; l0 < p.n_layers; l0 += 4) {
                const int nl = min(4, p.n_layers - l0);
                const uint64_t dV = tc_desc(sVr + (uint32_t)(t & 1) * kVBuf + (uint32_t)l0 * kTcTileK, kTcTileK);
                const uint32_t idO = tc_idesc(true, nl * kDh);
                const uint32_t acc = tmem + 64u + 64u * (uint32_t)l0;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {  // 16 keys per step: 32 bytes along a weight row, two 8-row groups of values
                    tc_mma(acc, dPh + 2 * ks, dV + 128 * ks, idO, (kc > 0 || ks > 0) ? 1u : 0u);
                    if (kTcRemainder) tc_mma(acc, dPl + 2 * ks, dV + 128 * ks, idO, 1u);
                }
            }
            tc_commit(bar_o);
        }
    }
    if (!dead) {                                  // the outputs of the last step
        mma_wait(bar_o, phase_o);
        __syncthreads();
        if (dead_s) dead = true;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (p.S && p.causal && qrow < len && !dead && part == 0) {   // keys beyond the tile's last chunk: never seen by a causal row
        float* Srow = p.S + (((long long)seq * p.H + h) * p.cap + qrow) * p.ld_s;
        for (int j = n_chunks * kTcChunk; j < len; ++j) Srow[j] = 0.f;
    }
    // ---- outputs: this thread's row of every layer's accumulator
    if (!dead) {
        for (int l = 0; l < p.n_layers; ++l) {      // this thread's 16 dims of the row
            float a[kTcCols1];
            tc_ld(t_lane + 64u + 64u * (uint32_t)l, a);
            if (qrow < len) {
                uint4* dst = reinterpret_cast<uint4*>(p.out + (long long)l * p.layer_elems + seq_off + (long long)qrow * row_elems + part * kTcCols1);
#pragma unroll
                for (int c = 0; c < kTcCols1 / 8; ++c)
                    dst[c] = make_uint4(full_pack(a[8 * c], a[8 * c + 1]), full_pack(a[8 * c + 2], a[8 * c + 3]),
                                        full_pack(a[8 * c + 4], a[8 * c + 5]), full_pack(a[8 * c + 6], a[8 * c + 7]));
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"((uint32_t)kTcCols) : "memory");
}

// More than half of an SM's shared memory, so that CTAs never share an SM: each takes all 512
// columns of tensor memory, and a second CTA would only sit in tcgen05.alloc until the first is done.
constexpr size_t full_tc5_smem_bytes() {
    constexpr size_t need = 1024 + 3 * (size_t)kTcTileQ + (4 + 2 * (size_t)kTcMaxLayers) * kTcTileK;
    return need > 116 * 1024 ? need : 116 * 1024;
}

}  // namespace san
