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

// One 16-byte piece per thread and beam: a tile is 1 KB (8 bf16 rows) of every beam.  Small tiles
// because rows are short (20-35 positions at sentence sizes): with 4 KB tiles a third of the
// threads had no piece (measured: 256 threads 0.53, 128 threads 0.61, 64 threads 0.65 of the copy
// bandwidth on 21-row panels; 0.98-1.0 on 256-row panels with any of them).
constexpr int kReorderThreads = 64;

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
    int unit_pieces;               // 16-byte pieces per unit of lens (a cached row)
    int fixed_pieces;              // > 0: every beam with lens > 0 moves this many pieces (AAN sums)
    int max_units;                 // limit of lens (row capacity)
    int tiles_per_panel;           // tiles covering the longest run the host allows
    int* err;
};

// grid = (tiles_per_panel * n_heads * n_sent, n_planes).  Thread t of tile k owns piece
// k * kReorderThreads + t of the (plane, sentence, head) panel in every beam: it loads the piece of each
// beam's parent, the CTA meets at a barrier, it stores.  The address arithmetic that does not
// depend on the beam is done once per thread; the copy itself is a handful of instructions
// per piece, so that the kernel is bound by HBM and not by instruction issue.
// BMAX: beams a thread keeps in registers (8 for the usual beams, SAN_MAX_BEAM for the widest).
template <int BMAX>
__global__ void __launch_bounds__(kReorderThreads) beam_reorder_kernel(const ReorderParams p) {
    unsigned u = blockIdx.x;
    const int tile = (int)(u % (unsigned)p.tiles_per_panel); u /= (unsigned)p.tiles_per_panel;
    const int h = (int)(u % (unsigned)p.n_heads);
    const int item = (int)(u / (unsigned)p.n_heads);
    const int plane = blockIdx.y;
    const int sent = p.sent_ids[item];
    const bool reporter = (plane == 0 && h == 0 && tile == 0 && threadIdx.x == 0);
    if (sent < 0 || sent >= p.max_sent) {                  // uniform over the CTA
        if (reporter) record_error(p.err, TAG_REORDER, item, sent, p.max_sent);
        return;
    }
    const int piece = tile * kReorderThreads + (int)threadIdx.x;
    char* panel = p.base + (long long)plane * p.plane_bytes + (long long)h * p.head_bytes +
                  (long long)sent * p.beam * p.seq_bytes + (long long)piece * 16;
    const int* parent = p.parent + item * p.beam;
    const int* lens = p.lens + item * p.beam;
    uint4 v[BMAX];
    unsigned take = 0;                                     // beams whose piece this thread moves
#pragma unroll
    for (int s = 0; s < BMAX; ++s) {
        if (s >= p.beam) break;
        const int par = parent[s], len = lens[s];
        if (par < 0 || par >= p.beam) { if (reporter) record_error(p.err, TAG_REORDER, item * p.beam + s, par, p.beam); continue; }
        if (len < 0 || len > p.max_units) { if (reporter) record_error(p.err, TAG_REORDER, item * p.beam + s, len, p.max_units); continue; }
        const int pieces = p.fixed_pieces > 0 ? (len > 0 ? p.fixed_pieces : 0) : len * p.unit_pieces;
        if (par == s || piece >= pieces) continue;         // keeps its own history / beyond the rows taken
        v[s] = ld16_once(panel + par * p.seq_bytes);
        take |= 1u << s;
    }
    __syncthreads();            // every piece of the tile that is needed has been read
#pragma unroll
    for (int s = 0; s < BMAX; ++s)
        if (take & (1u << s)) *reinterpret_cast<uint4*>(panel + s * p.seq_bytes) = v[s];
}

}  // namespace san
