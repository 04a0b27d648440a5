// Beam-search cache reorder (Section 4.1 decodes with beam search: after each step every
// surviving hypothesis continues the cache of the parent it extends).
//
// For every self-attention plane (keys of block-first layers, values of every layer) beam s
// of a sentence takes over the first lens[s] cached rows of beam parent[s] of the SAME
// sentence; with AAN in place of self-attention it takes over the parent's running sum.
// The gather is done in place.  That is safe because a hypothesis only ever descends from a
// hypothesis of its own sentence: a CTA owns one tile = the same run of positions of one
// (plane, sentence, head) in all beams, loads every 16-byte piece it needs into registers,
// meets at a barrier, and only then stores; no other CTA reads or writes that tile.  Rows keep
// their position, so the chunk permutation of bf16 rows (a function of the position alone)
// is preserved by a bit copy.  Beams that keep their own history (parent == self) move
// nothing.  HBM-bound: 2 x 16 bytes per piece moved, nothing else.
#pragma once

#include "san_kernels.cuh"

namespace san {

constexpr int kReorderThreads = 256;
constexpr int kReorderPieces = 4;                                      // 16-byte pieces per thread
constexpr int kReorderTile = kReorderThreads * kReorderPieces;         // pieces per tile, all beams together

// The tile is written later in the same kernel, so the read-only (non-coherent) path is not
// allowed here: an ordinary load, kept out of L1 because every piece is read once.
__device__ __forceinline__ uint4 ld16_once(const void* p) {
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

struct ReorderParams {
    char* base;                    // plane 0
    long long plane_bytes;         // between planes
    long long seq_bytes;           // between the sequences (beams) of a plane
    long long head_bytes;          // between the heads of a sequence (unused when n_heads == 1)
    const int* sent_ids; const int* parent; const int* lens;    // [n_sent], [n_sent][beam], [n_sent][beam]
    int n_planes, n_sent, n_heads, beam, max_sent;
    int unit_bytes;                // bytes per unit of lens (a cached row)
    int fixed_bytes;               // > 0: every beam with lens > 0 moves this many bytes (AAN sums)
    int max_units;                 // limit of lens (row capacity)
    int tiles_per_panel;           // tiles covering the longest run the host allows
    int* err;
};

// grid = n_planes * n_sent * n_heads * tiles_per_panel CTAs
static __global__ void __launch_bounds__(kReorderThreads) beam_reorder_kernel(const ReorderParams p) {
    unsigned u = blockIdx.x;
    const int tile = (int)(u % (unsigned)p.tiles_per_panel); u /= (unsigned)p.tiles_per_panel;
    const int h = (int)(u % (unsigned)p.n_heads); u /= (unsigned)p.n_heads;
    const int item = (int)(u % (unsigned)p.n_sent);
    const int plane = (int)(u / (unsigned)p.n_sent);
    const int per_beam = kReorderTile / p.beam;            // pieces of one beam in a tile
    const int sent = p.sent_ids[item];
    const bool reporter = (plane == 0 && h == 0 && tile == 0);
    const bool sent_ok = sent >= 0 && sent < p.max_sent;
    if (!sent_ok && reporter && threadIdx.x == 0) record_error(p.err, TAG_REORDER, item, sent, p.max_sent);

    uint4 v[kReorderPieces];
    char* dst[kReorderPieces];
#pragma unroll
    for (int r = 0; r < kReorderPieces; ++r) {
        dst[r] = nullptr;
        const int e = r * kReorderThreads + (int)threadIdx.x;      // consecutive threads: consecutive pieces of a beam
        const int s = e / per_beam, k = e - s * per_beam;
        if (!sent_ok || s >= p.beam) continue;
        const int par = p.parent[item * p.beam + s], len = p.lens[item * p.beam + s];
        if (par < 0 || par >= p.beam) { if (reporter && k == 0) record_error(p.err, TAG_REORDER, item * p.beam + s, par, p.beam); continue; }
        if (len < 0 || len > p.max_units) { if (reporter && k == 0) record_error(p.err, TAG_REORDER, item * p.beam + s, len, p.max_units); continue; }
        if (par == s) continue;                                    // keeps its own history
        const long long bytes = p.fixed_bytes > 0 ? (len > 0 ? (long long)p.fixed_bytes : 0) : (long long)len * p.unit_bytes;
        const long long off = ((long long)tile * per_beam + k) * 16;
        if (off >= bytes) continue;
        char* panel = p.base + (long long)plane * p.plane_bytes + (long long)h * p.head_bytes + off;
        v[r] = ld16_once(panel + ((long long)sent * p.beam + par) * p.seq_bytes);
        dst[r] = panel + ((long long)sent * p.beam + s) * p.seq_bytes;
    }
    __syncthreads();            // every piece of the tile that is needed has been read
#pragma unroll
    for (int r = 0; r < kReorderPieces; ++r)
        if (dst[r]) *reinterpret_cast<uint4*>(dst[r]) = v[r];
}

}  // namespace san
