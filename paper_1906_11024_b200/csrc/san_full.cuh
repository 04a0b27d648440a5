// Full-sequence shared attention (the encoder-side use of Table 5, and decoder prefill):
// for every sequence and head the l x l weights S = Softmax(Q.K^T / sqrt(64)) are computed
// once, by the lowest layer of a block (Eq. 1, Eq. 3), and applied to the values of every
// layer of the block (Eq. 2, Eq. 4).  Unlike the decode step this is a dense contraction
// (l queries against l keys), so it runs on the tensor cores (mma.sync m16n8k16, bf16
// operands, float32 accumulate).
//
// CTA = (tile of 64 queries, head, sequence), four warps of 16 query rows each.
//   1. scores: key rows stream through shared memory in chunks of 64; a warp multiplies its
//      16 x 64 query fragment (registers) with the chunk and writes the 16 x 64 scores into its
//      strip of shared memory (float32, one row per query, all l keys).
//   2. softmax over each strip row (max, exp2, sum, divide); the normalised weights stay in
//      the strip and are written to S for the caller if wanted.
//   3. apply, layer by layer: value rows stream through shared memory in chunks of 64; the
//      weights are read from the strip as a bf16 high part plus a bf16 remainder (two MMAs, so
//      that they keep about 16 bits) and multiplied with the chunk read through
//      ldmatrix.trans.  S is computed once however many layers the block has.
#pragma once

#include "san_kernels.cuh"

namespace san {

constexpr int kFullQ = 64;            // queries per CTA
constexpr int kFullChunk = 64;        // keys per shared-memory chunk
constexpr int kFullRowBytes = 144;    // a 64-element bf16 row padded by 16 bytes: conflict-free for both access patterns
constexpr int kFullMaxLen = 512;      // keys a strip holds at most

struct FullParams {
    const __nv_bfloat16* q; const __nv_bfloat16* k; const __nv_bfloat16* v;   // [n_seq][cap][H][64]; v: [n_layers] of those
    __nv_bfloat16* out;                                                       // [n_layers][n_seq][cap][H][64]
    float* S; long long ld_s;                                                 // [n_seq][H][cap][ld_s] or null
    const int* lens;
    long long layer_elems;         // elements between layers in v and out
    int n_seq, H, cap, max_len, n_layers, causal, strip_ld;                   // strip_ld: floats per strip row (sized for max_len)
    float scale_log2e;
};

__device__ __forceinline__ void full_mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t full_pack(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// A chunk = 64 rows of 64 bf16 (row stride H*64 elements in global memory).  Its 512 pieces
// of 16 bytes are fetched into registers, four per thread, one chunk ahead of their use, and
// stored into the padded shared-memory chunk when the previous chunk has been consumed; rows
// at or beyond `rows` read as zero.
__device__ __forceinline__ void full_fetch(uint4 (&pre)[4], const __nv_bfloat16* src, long long row_elems, int rows) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int u = (int)threadIdx.x + i * 128, r = u >> 3, c = u & 7;
        pre[i] = r < rows ? ld16_stream(src + (long long)r * row_elems + c * 8) : make_uint4(0, 0, 0, 0);
    }
}
__device__ __forceinline__ void full_store(unsigned char* chunk, const uint4 (&pre)[4]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int u = (int)threadIdx.x + i * 128, r = u >> 3, c = u & 7;
        *reinterpret_cast<uint4*>(chunk + r * kFullRowBytes + c * 16) = pre[i];
    }
}

extern __shared__ __align__(16) unsigned char full_smem[];

static __global__ void __launch_bounds__(128, 4) full_block_kernel(const FullParams p) {
    const int seq = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * kFullQ;
    const int len = min(p.lens[seq], p.max_len);       // the strips are sized for max_len: longer sequences are cut there
    if (q0 >= len) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gid = lane >> 2, tig = lane & 3;
    const long long row_elems = (long long)p.H * kDh;
    const long long seq_off = ((long long)seq * p.cap) * row_elems + (long long)h * kDh;
    unsigned char* chunk = full_smem;                                                   // kFullChunk padded rows
    float* strip = reinterpret_cast<float*>(full_smem + kFullChunk * kFullRowBytes) + (long long)warp * 16 * p.strip_ld;
    const int qa = q0 + warp * 16 + gid, qb = qa + 8;                                    // this lane's two query rows
    const int n_keys = p.causal ? min(len, q0 + kFullQ) : len;                           // keys any query of the tile sees
    const int n_chunks = (n_keys + kFullChunk - 1) / kFullChunk;
    const int n_pad = (n_keys + 15) & ~15;             // keys that are scored, normalised and applied: whole 16-key MMA blocks

    // the first key chunk is on its way while the query fragments are read
    uint4 pre[4];
    full_fetch(pre, p.k + seq_off, row_elems, min(kFullChunk, len));

    // query fragments (A operand, 16 queries x 64 dims): rows beyond the sequence read as zero
    uint32_t qf[4][4];
    {
        const __nv_bfloat16* qr_a = p.q + seq_off + (long long)qa * row_elems;
        const __nv_bfloat16* qr_b = p.q + seq_off + (long long)qb * row_elems;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            qf[ks][0] = qa < len ? *reinterpret_cast<const uint32_t*>(qr_a + 16 * ks + 2 * tig) : 0u;
            qf[ks][1] = qb < len ? *reinterpret_cast<const uint32_t*>(qr_b + 16 * ks + 2 * tig) : 0u;
            qf[ks][2] = qa < len ? *reinterpret_cast<const uint32_t*>(qr_a + 16 * ks + 2 * tig + 8) : 0u;
            qf[ks][3] = qb < len ? *reinterpret_cast<const uint32_t*>(qr_b + 16 * ks + 2 * tig + 8) : 0u;
        }
    }
    const int vrow_l = (lane & 7) + ((lane >> 3) & 1) * 8;          // ldmatrix.trans: key row this lane addresses in a 16-key block
    const int vcol_l = (lane >> 4) * 8;                             // and its dim offset inside a pair of 8-dim tiles
    const uint32_t chunk_s = (uint32_t)__cvta_generic_to_shared(chunk);
    float acc[8][4];

    // Panels in order: the keys, then the values of each layer; every panel in chunks of 64 rows.
    // panel 0 fills the strip with scores and ends with the softmax; panel l+1 applies the strip
    // to layer l's values and ends with that layer's output.
    for (int panel = 0; panel <= p.n_layers; ++panel) {
        for (int kc = 0; kc < n_chunks; ++kc) {
            const int k0 = kc * kFullChunk;
            __syncthreads();                                   // every warp is done with the previous chunk
            full_store(chunk, pre);
            __syncthreads();
            {   // fetch the chunk after this one
                int np = panel, nkc = kc + 1;
                if (nkc == n_chunks) { np += 1; nkc = 0; }
                if (np <= p.n_layers) {
                    const __nv_bfloat16* base = np == 0 ? p.k : p.v + (long long)(np - 1) * p.layer_elems;
                    full_fetch(pre, base + seq_off + (long long)nkc * kFullChunk * row_elems, row_elems,
                               min(kFullChunk, len - nkc * kFullChunk));
                }
            }
            if (panel == 0) {
                // ---- scores (log2 domain) into the strip; masked keys get -inf
#pragma unroll
                for (int nt = 0; nt < kFullChunk / 8; ++nt) {      // 8 keys per MMA
                    if (k0 + nt * 8 >= n_pad) break;
                    float sc[4] = {0.f, 0.f, 0.f, 0.f};
                    const unsigned char* krow = chunk + (nt * 8 + gid) * kFullRowBytes + 4 * tig;     // key nt*8+gid, dims 2tig..
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        const uint32_t b0 = *reinterpret_cast<const uint32_t*>(krow + 32 * ks);
                        const uint32_t b1 = *reinterpret_cast<const uint32_t*>(krow + 32 * ks + 16);
                        full_mma(sc, qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b0, b1);
                    }
                    const int key = k0 + nt * 8 + 2 * tig;         // sc[0], sc[1]: query qa, keys key, key+1; sc[2], sc[3]: query qb
                    float2 za, zb;
                    za.x = (key < len && (!p.causal || key <= qa)) ? sc[0] * p.scale_log2e : -INFINITY;
                    za.y = (key + 1 < len && (!p.causal || key + 1 <= qa)) ? sc[1] * p.scale_log2e : -INFINITY;
                    zb.x = (key < len && (!p.causal || key <= qb)) ? sc[2] * p.scale_log2e : -INFINITY;
                    zb.y = (key + 1 < len && (!p.causal || key + 1 <= qb)) ? sc[3] * p.scale_log2e : -INFINITY;
                    *reinterpret_cast<float2*>(strip + gid * p.strip_ld + key) = za;
                    *reinterpret_cast<float2*>(strip + (gid + 8) * p.strip_ld + key) = zb;
                }
                if (kc + 1 < n_chunks) continue;
                // ---- softmax of the warp's 16 rows over the scored keys [0, n_pad): eight lanes per
                // row, four rows side by side (lane i of a row takes keys i, i + 8, ...: with a row
                // stride of 8 mod 32 words the 32 lanes touch 32 different banks)
                __syncwarp();
                const int sub = lane & 7;
#pragma unroll
                for (int rg = 0; rg < 4; ++rg) {
                    const int r = rg * 4 + (lane >> 3);
                    float* row = strip + r * p.strip_ld;
                    const int qrow = q0 + warp * 16 + r;
                    float m = -INFINITY;
                    for (int j = sub; j < n_pad; j += 8) m = fmaxf(m, row[j]);
#pragma unroll
                    for (int o = 4; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
                    if (qrow >= len) m = 0.f;                  // a row outside the sequence is never stored; keep it finite
                    float s = 0.f;
                    for (int j = sub; j < n_pad; j += 8) { const float e = exp2f(row[j] - m); row[j] = e; s += e; }
#pragma unroll
                    for (int o = 4; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                    const float inv = s > 0.f ? 1.0f / s : 0.f;
                    float* Srow = (p.S && qrow < len) ? p.S + (((long long)seq * p.H + h) * p.cap + qrow) * p.ld_s : nullptr;
                    for (int j = sub; j < n_pad; j += 8) {
                        const float w = row[j] * inv;
                        row[j] = w;
                        if (Srow && j < len) Srow[j] = w;      // masked keys of a causal row are stored as 0
                    }
                    if (Srow && p.causal) for (int j = n_pad + sub; j < len; j += 8) Srow[j] = 0.f;
                }
                __syncwarp();
                continue;
            }
            // ---- apply the strip to this chunk of the layer's values
            if (kc == 0) {
#pragma unroll
                for (int x = 0; x < 8; ++x)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[x][e] = 0.f;
            }
#pragma unroll
            for (int kb = 0; kb < kFullChunk; kb += 16) {           // 16 keys per MMA
                if (k0 + kb >= n_pad) break;
                // A = weights of queries (gid, gid+8) at keys k0+kb + {2tig, 2tig+1, 2tig+8, 2tig+9}
                const float2 wa0 = *reinterpret_cast<const float2*>(strip + gid * p.strip_ld + k0 + kb + 2 * tig);
                const float2 wb0 = *reinterpret_cast<const float2*>(strip + (gid + 8) * p.strip_ld + k0 + kb + 2 * tig);
                const float2 wa1 = *reinterpret_cast<const float2*>(strip + gid * p.strip_ld + k0 + kb + 2 * tig + 8);
                const float2 wb1 = *reinterpret_cast<const float2*>(strip + (gid + 8) * p.strip_ld + k0 + kb + 2 * tig + 8);
                const uint32_t h0 = full_pack(wa0.x, wa0.y), h1 = full_pack(wb0.x, wb0.y);
                const uint32_t h2 = full_pack(wa1.x, wa1.y), h3 = full_pack(wb1.x, wb1.y);
                const uint32_t r0 = full_pack(wa0.x - __uint_as_float(h0 << 16), wa0.y - __uint_as_float(h0 & 0xffff0000u));
                const uint32_t r1 = full_pack(wb0.x - __uint_as_float(h1 << 16), wb0.y - __uint_as_float(h1 & 0xffff0000u));
                const uint32_t r2 = full_pack(wa1.x - __uint_as_float(h2 << 16), wa1.y - __uint_as_float(h2 & 0xffff0000u));
                const uint32_t r3 = full_pack(wb1.x - __uint_as_float(h3 << 16), wb1.y - __uint_as_float(h3 & 0xffff0000u));
#pragma unroll
                for (int dp = 0; dp < 4; ++dp) {                    // a pair of 8-dim tiles per ldmatrix
                    uint32_t b[4];
                    const uint32_t addr = chunk_s + (uint32_t)((kb + vrow_l) * kFullRowBytes + (dp * 16 + vcol_l) * 2);
                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3]) : "r"(addr) : "memory");
                    full_mma(acc[2 * dp], h0, h1, h2, h3, b[0], b[1]);
                    full_mma(acc[2 * dp], r0, r1, r2, r3, b[0], b[1]);
                    full_mma(acc[2 * dp + 1], h0, h1, h2, h3, b[2], b[3]);
                    full_mma(acc[2 * dp + 1], r0, r1, r2, r3, b[2], b[3]);
                }
            }
            if (kc + 1 < n_chunks) continue;
            // acc[x][0], [1]: query qa, dims 8x + 2tig, +1; acc[x][2], [3]: query qb
            const long long lo = (long long)(panel - 1) * p.layer_elems + seq_off + 2 * tig;
            __nv_bfloat16* oa = p.out + lo + (long long)qa * row_elems;
            __nv_bfloat16* ob = p.out + lo + (long long)qb * row_elems;
#pragma unroll
            for (int x = 0; x < 8; ++x) {
                if (qa < len) *reinterpret_cast<uint32_t*>(oa + 8 * x) = full_pack(acc[x][0], acc[x][1]);
                if (qb < len) *reinterpret_cast<uint32_t*>(ob + 8 * x) = full_pack(acc[x][2], acc[x][3]);
            }
        }
    }
}

}  // namespace san
