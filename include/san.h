/*
 * san.h -- C ABI of the shared-attention (SAN) decode library for NVIDIA B200 (sm_100a).
 *
 * The library implements the cached attention of auto-regressive Transformer decoding
 * when attention weights are shared inside blocks of adjacent decoder layers
 * ("Sharing Attention Weights for Fast Transformer", arXiv 1906.11024).
 *
 * Notation follows the paper: S = Softmax(Q.K^T / sqrt(d_k)) are the attention WEIGHTS
 * (Eq. 1) and the attention OUTPUT is S.V (Eq. 2; the paper calls it A, this header calls
 * it O).  In a block of pi adjacent layers only the lowest layer m computes S^m from its
 * own queries and keys; layers m+1 .. m+pi-1 reuse S^m and apply it to their own values
 * (Eq. 3-4).  Hence only block-first layers keep a key cache (Section 3.2, memory note).
 *
 * General rules
 *  - Every function returns a status (SAN_OK = 0).  Nothing throws or traps, and no kernel
 *    waits on another kernel, CTA or rank.  The only device-side waits are a CTA's waits for
 *    its OWN asynchronous copies or tensor-core operations (mbarrier waits in the kernels
 *    behind san_decode_step and san_full_block); each gives up after about a second, makes
 *    the kernel stop early.  san_decode_step reports it as SAN_ERR_TIMEOUT through
 *    san_device_status, which then also clears the context's split-row tickets so that later
 *    steps start clean; san_full_block has no status word, and a tile whose wait ran out
 *    leaves its output rows unwritten.
 *  - All `d_` pointers are DEVICE pointers owned by the caller; all others are HOST
 *    pointers.  The library allocates no device memory: the cache arena and the
 *    workspace are caller buffers handed to san_create.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  No hot call
 *    synchronises the host.  Calls on one context must be ordered on the device (same
 *    stream, or events between streams): they share the context's workspace.
 *  - Host-checkable mistakes (null pointers, shapes, an invalid policy, a layer outside
 *    the block, capacity) are reported before anything is launched.  Mistakes visible
 *    only on the device (an id out of range, a length < 1 or beyond capacity) make the
 *    kernel skip that item and record the first such error in a device word, read back
 *    with san_device_status.
 *  - Element type is SAN_F32 or SAN_BF16 for q/k/v/x/outputs; S is always float32;
 *    products, sums and the softmax are float32.  d_head must be 64.
 *  - Sequences are numbered 0 .. max_sent*beam-1; sequence s belongs to sentence
 *    s / beam (the beams of a sentence read the same encoder memory, Section 2).
 *
 * Cache layout inside the arena (head-major; every (id, head) panel is contiguous and
 * each row is 64 elements = 128 B bf16 / 256 B f32, 16-byte aligned).  bf16 rows are stored
 * with their eight 16-byte chunks permuted: chunk c of the row at position pos sits at chunk
 * c ^ (pos & 7), so that a tile of rows copied verbatim into shared memory can be read eight
 * rows at a time without bank conflicts; callers never see this unless they read the arena
 * directly.  float32 rows are stored in natural order.
 *    self K   [self block ][sequence][head][max_tgt_len][64]   (block-first layers only)
 *    self V   [layer      ][sequence][head][max_tgt_len][64]
 *    memory K [encdec block][sentence][head][max_src_len][64]
 *    memory V [layer       ][sentence][head][max_src_len][64]  (one plane per BLOCK when
 *                                                               encdec_shared_context)
 *    AAN sum  [layer][sequence][n_heads*64] float32             (only when self_is_aan)
 */
#ifndef SAN_H_
#define SAN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct san_ctx san_ctx; /* opaque; lives in host memory */

enum {
    SAN_OK = 0,
    SAN_ERR_NULL = 1,         /* a required pointer is NULL */
    SAN_ERR_SHAPE = 2,        /* a size or count is out of range */
    SAN_ERR_POLICY = 3,       /* block sizes / block map do not describe a valid policy */
    SAN_ERR_CAPACITY = 4,     /* a caller buffer is too small, or more blocks than key planes */
    SAN_ERR_DTYPE = 5,
    SAN_ERR_RANGE = 6,        /* layer/block/position outside what the policy or config allows */
    SAN_ERR_CUDA = 7,         /* a CUDA runtime call failed (launch configuration, bad stream...) */
    SAN_ERR_DEVICE_CHECK = 8, /* a kernel met an invalid id/length/position and skipped the item */
    SAN_ERR_TIMEOUT = 9,      /* a kernel's bounded wait for its own copies ran out (see General rules) */
    SAN_ERR_UNSUPPORTED = 10
};
enum { SAN_F32 = 0, SAN_BF16 = 1 };
enum { SAN_SELF = 0, SAN_ENCDEC = 1 };

#define SAN_MAX_LAYERS 64
#define SAN_MAX_BEAM 32

typedef struct {
    int32_t n_layers;    /* M, 1..SAN_MAX_LAYERS */
    int32_t n_heads;     /* H */
    int32_t d_head;      /* must be 64 */
    int32_t max_sent;    /* sentences the caches have room for */
    int32_t beam;        /* sequences per sentence, 1..SAN_MAX_BEAM */
    int32_t max_tgt_len; /* self-attention cache rows per sequence */
    int32_t max_src_len; /* encoder-memory rows per sentence */
    int32_t dtype;       /* SAN_F32 or SAN_BF16 */
    int32_t self_is_aan; /* 1: decoder self-attention is the cumulative average (san_aan_step) */
    int32_t encdec_shared_context; /* 1: Eq. 5, one O (and one V plane) per enc-dec block */
} san_config;

/* Bytes the caller must provide for a configuration whose self / enc-dec policies have
 * n_self_blocks / n_encdec_blocks blocks (the key-cache planes; Section 3.2: layers that
 * take their weights from another layer keep no keys).  Either output may be NULL. */
int32_t san_query_bytes(const san_config* cfg, int32_t n_self_blocks, int32_t n_encdec_blocks,
                        size_t* cache_bytes, size_t* workspace_bytes);

/* Creates a context over caller-owned device buffers (256-byte aligned).  The sharing
 * policies are given as block sizes {pi_1..pi_N} bottom-up (Section 3.3); their block
 * counts fix the number of key planes carved out of the arena.  Zeroes the workspace
 * header on the default stream and waits for it (the one synchronising call besides
 * san_device_status).  The arena is not cleared. */
int32_t san_create(const san_config* cfg, const int32_t* self_sizes, int32_t n_self,
                   const int32_t* encdec_sizes, int32_t n_encdec, void* d_cache, size_t cache_bytes,
                   void* d_workspace, size_t workspace_bytes, san_ctx** out);
int32_t san_destroy(san_ctx* ctx);

/* Sharing policy (Section 3.3): block sizes bottom-up with sum = n_layers and every size
 * >= 1, or the same thing as a per-layer block id (starts at 0; each next layer keeps the
 * id or raises it by one).  A policy with more blocks than the context has key planes is
 * refused with SAN_ERR_CAPACITY.  Changing the policy does not move cached rows. */
int32_t san_policy_set_sizes(san_ctx* ctx, int32_t kind, const int32_t* sizes, int32_t n_blocks);
int32_t san_policy_set_map(san_ctx* ctx, int32_t kind, const int32_t* block_of_layer, int32_t n_layers);
/* Any output may be NULL.  block_of_layer[n_layers], first_layer_of_block[n_blocks]. */
int32_t san_policy_get_map(const san_ctx* ctx, int32_t kind, int32_t* block_of_layer,
                           int32_t* first_layer_of_block, int32_t* n_blocks);

/* Attention cache (Section 4.1 uses one; Section 2: enc-dec keys/values come from the
 * encoder output).  Copies new rows into the caches of layers [layer_begin, layer_end):
 *   kind = SAN_SELF   d_ids = sequence ids, rows go to the self-attention K/V caches;
 *   kind = SAN_ENCDEC d_ids = sentence ids, rows go to the encoder-memory K/V.
 * Item i writes d_nrows[i] rows (1 if d_nrows is NULL) starting at row d_pos[i] (0 if
 * d_pos is NULL).  Source layout, `rows_per_item` = row capacity of one item (>= every
 * d_nrows[i]; 1 for a decode step):
 *   d_v_new [layers in range          ][n_items][rows_per_item][H][64]
 *   d_k_new [block-first layers in range][n_items][rows_per_item][H][64]   (in layer order)
 * d_k_new must be NULL iff the range holds no block-first layer.  With
 * encdec_shared_context only block-first layers may be in an ENCDEC range.
 * Not allowed for SAN_SELF when self_is_aan.  Payload is copied bit for bit. */
int32_t san_cache_append(san_ctx* ctx, int32_t kind, int32_t layer_begin, int32_t layer_end,
                         const void* d_k_new, const void* d_v_new, const int32_t* d_ids,
                         const int32_t* d_pos, const int32_t* d_nrows, int32_t n_items,
                         int32_t rows_per_item, void* stream);

/* Eq. 1 for one decode step, at the lowest layer of `block` (Eq. 3):
 *   S[j] = exp(z_j - max z) / sum_j exp(z_j - max z),  z_j = (q . K_j) / sqrt(64),
 * over cached rows j in [0, d_lens[i]).
 *   kind = SAN_SELF    d_ids sequence ids; d_q [n_items][H][64]; d_S [n_items][H][ld_s]
 *   kind = SAN_ENCDEC  d_ids sentence ids; d_q [n_items][beam][H][64];
 *                      d_S [n_items][beam][H][ld_s]; d_lens[i] = source length; every
 *                      key tile is read once for all beams of the sentence.
 * max_len is a host-side upper bound on d_lens (1..capacity; 0 = capacity) used to size
 * the launch; a longer length is a device-check error.  ld_s >= max_len.  Entries of a
 * row beyond its length are left untouched.  Long rows are split over several warps
 * (partial max/sum in the workspace, combined by the last warp to finish; nothing waits). */
int32_t san_attn_weights(san_ctx* ctx, int32_t kind, int32_t block, const void* d_q,
                         const int32_t* d_ids, const int32_t* d_lens, int32_t n_items,
                         int32_t max_len, float* d_S, int64_t ld_s, void* stream);

/* Eq. 2 with Eq. 4: for every layer l in [layer_begin, layer_end), all inside `block`,
 *   O_l = sum_{j in [p0, p1)} S[j] * V_l[j]
 * with the block's weights S (layout as written by san_attn_weights) and each layer's own
 * cached values, in one launch; S is staged on chip once per work item and reused for
 * every layer.  p0 = d_pos_begin[i] (0 if NULL), p1 = d_pos_end[i].
 *   d_out [layer_end-layer_begin][n_items]([beam])[H][64], element type = cfg.dtype
 *         (rounded to nearest even from float32 for bf16).
 * accumulate != 0 adds to what d_out holds (for finishing a layer whose newest value row
 * arrived after the block's history was applied).  With encdec_shared_context (Eq. 5) an
 * ENCDEC call must name exactly the block's first layer; the one output serves the block.
 * max_len bounds d_pos_end as in san_attn_weights. */
int32_t san_attn_apply(san_ctx* ctx, int32_t kind, int32_t block, int32_t layer_begin,
                       int32_t layer_end, const float* d_S, int64_t ld_s, const int32_t* d_ids,
                       const int32_t* d_pos_begin, const int32_t* d_pos_end, int32_t n_items,
                       int32_t max_len, void* d_out, int32_t accumulate, void* stream);

/* Average attention in place of decoder self-attention (the AAN model the paper combines
 * with SAN in Table 6): for layers [layer_begin, layer_end) and item i with sequence
 * d_ids[i] at 1-based target position d_t[i]:
 *   sum_l[seq] += x_l[i];  out_l[i] = sum_l[seq] / d_t[i]      (mean of positions 1..t)
 * d_t[i] == 1 restarts the sum from x.  d_x, d_out: [layers in range][n_items][H*64]. */
int32_t san_aan_step(san_ctx* ctx, int32_t layer_begin, int32_t layer_end, const void* d_x,
                     const int32_t* d_ids, const int32_t* d_t, int32_t n_items, void* d_out,
                     void* stream);

/* Forget the history of the listed sequences under average attention (Table 6 pairing): the
 * running sums of every layer are set to zero for each sequence d_seq_ids[i], i < n, so that
 * a cache slot can be handed to another hypothesis or sentence at any point of its count.
 * After the call the next san_aan_step at position t returns x / t for such a sequence, as
 * if its earlier inputs had been zero; restarting the count at t = 1 needs no reset (that
 * step overwrites the sum).  Only for contexts with self_is_aan (else SAN_ERR_UNSUPPORTED).
 * An id outside 0 .. max_sent*beam-1 is skipped and reported through san_device_status. */
int32_t san_seq_reset(san_ctx* ctx, const int32_t* d_seq_ids, int32_t n, void* stream);

/* One whole decode step in ONE launch: for every block of both attention kinds, append
 * this step's rows (Section 4.1 cache), compute the block's weights at its lowest layer
 * (Eq. 1, Eq. 3) and apply them to the values of every layer of the block (Eq. 2, Eq. 4;
 * Eq. 5 with encdec_shared_context); with self_is_aan the cumulative average replaces
 * the self-attention part.  Same arithmetic and outputs as the sequence
 *     san_cache_append(SELF, 0..M) ; per block san_attn_weights + san_attn_apply
 * for inputs laid out for all layers at once (a caller that has every layer's q/k/v of
 * the step up front, e.g. a benchmark or a speculative/batched front end):
 *   d_q_self, d_k_new [n_self_blocks][n_seqs][H][64]   rows of the block-first layers
 *   d_v_new           [n_layers][n_seqs][H][64]
 *   d_seq_ids, d_pos  sequence ids and the row each writes this step (length = pos + 1)
 *   d_S_self          [n_self_blocks][n_seqs][H][ld_t] float32, or NULL if not wanted
 *   d_O_self          [n_layers][n_seqs][H][64]
 *   d_q_enc           [n_encdec_blocks][n_sent][beam][H][64]
 *   d_sent_ids, d_src_lens   sentence ids and their source lengths
 *   d_S_enc           [n_encdec_blocks][n_sent*beam][H][ld_s] float32, or NULL
 *   d_O_enc           [n_layers (or n_encdec_blocks with Eq. 5)][n_sent*beam][H][64]
 *   d_x_aan, d_t      [n_layers][n_seqs][H*64] and 1-based positions (self_is_aan only;
 *                     the averages go to d_O_self)
 * n_seqs == 0 skips the self/AAN part, n_sent == 0 the enc-dec part.  max_len / max_src
 * are host bounds on pos+1 / source lengths (0 = capacity).  Rows longer than the on-chip
 * score buffer are split into at most 32 spans; a bound that would need more returns
 * SAN_ERR_UNSUPPORTED (use the separate calls).  The kernel's waits on its own copies are
 * bounded: if one runs out the step reports SAN_ERR_TIMEOUT through san_device_status.  A beam
 * wider than 8 takes one launch per group of 8 query rows. */
typedef struct {
    const void* d_q_self; const void* d_k_new; const void* d_v_new;
    const int32_t* d_seq_ids; const int32_t* d_pos; int32_t n_seqs; int32_t max_len;
    float* d_S_self; int64_t ld_t; void* d_O_self;
    const void* d_q_enc; const int32_t* d_sent_ids; const int32_t* d_src_lens; int32_t n_sent; int32_t max_src;
    float* d_S_enc; int64_t ld_s; void* d_O_enc;
    const void* d_x_aan; const int32_t* d_t;
} san_step_args;
int32_t san_decode_step(san_ctx* ctx, const san_step_args* args, void* stream);

/* Which kernel san_decode_step launches, and (for testing and tuning) how its rows are cut.
 * The library has three implementations of the one-launch step (same arithmetic, Eq. 1-5):
 *   which = 1  per-warp pipeline: every warp streams the tiles of its own row (float32 and bf16);
 *   which = 2  team pipeline (bf16): four producer warps each stream bundles of two units to a team
 *              of two warps, a unit being up to four heads of one sequence or one of two spans of
 *              a long row; SAN_ERR_UNSUPPORTED from the step if a shape does not fit;
 *   which = 3  short rows (bf16, max_len and max_src at most 96): a warp fetches whole planes of 1, 2
 *              or 4 heads (heads_per_unit; fewer where they would not fit its ring) and keeps the
 *              scores in registers; layers_per_unit as below; SAN_ERR_UNSUPPORTED from the step
 *              if the bounds are larger;
 *   which = 0  automatic (the default): the team pipeline for steps whose rows are long enough to be
 *              split over the warps of a team, the short-rows kernel for launches that hold
 *              encoder-decoder attention alone (where each measured faster), else the per-warp one.
 * A value may carry a second one for encoder-decoder attention in its bits 8 and up, as (v + 1) << 8.
 * spans_log2 >= 0 overrides the automatic cut of the team pipeline: every row is dealt to
 * 1 << spans_log2 warps (0..1); with one span up to heads_per_unit (1, 2 or 4) heads of one
 * sequence or sentence go to a warp where the head count allows (at most 2 where several
 * beams share a key tile); tiles hold tile_pos positions (a multiple of 16);
 * layers_per_unit > 0 caps the layers one warp applies (the block's other layers go to
 * further warps, which recompute S); grab_mult >= 1 makes the bundles shrink earlier towards
 * the end of the launch.  spans_log2 < 0 restores the automatic cut. */
int32_t san_step_kernel_select(san_ctx* ctx, int32_t which, int32_t spans_log2, int32_t heads_per_unit,
                               int32_t tile_pos, int32_t layers_per_unit, int32_t grab_mult);

/* Which kernel the last san_decode_step of this context launched (1, 2 or 3 as above, 0 before the
 * first step) and, for the team pipeline and the short-rows kernel, how many heads of one sequence / sentence it gave
 * to one warp: rows_per_unit[0] for self-attention, [1] for encoder-decoder attention (may
 * be NULL).  For tests and benchmarks that must know what they measured. */
int32_t san_step_kernel_used(const san_ctx* ctx, int32_t* which, int32_t* rows_per_unit);

/* san_decode_step for a caller whose step inputs and outputs live in HOST memory (pinned
 * memory if the copies are to overlap anything): the same step (Eq. 1-5, Section 4.1) with
 * the transfers issued by the library on `stream`, in order: every input array named in
 * `host` is copied into the array of the same field in `dev`, san_decode_step(ctx, dev) is
 * launched, then O_self and O_enc (and S_self / S_enc where both structs name a buffer) are
 * copied back into `host`.  `dev` is a complete argument block of caller-owned device
 * buffers and carries the counts, bounds and leading dimensions; the pointer fields of
 * `host` are HOST pointers of the same shapes (its scalar fields are ignored).  Nothing is
 * allocated and the host is not synchronised: `host` outputs are valid once `stream` has
 * reached this point, and `host` inputs must stay untouched until then. */
int32_t san_decode_step_host(san_ctx* ctx, const san_step_args* host, const san_step_args* dev, void* stream);

/* Beam-search cache reorder (Section 4.1: decoding runs a beam of hypotheses per sentence;
 * after a step each surviving hypothesis continues the attention cache of the hypothesis it
 * extends).  For item i = sentence d_sent_ids[i] and beam slot s, the sequence
 * sentence*beam + s takes over the first d_lens[i*beam + s] cached rows of the sequence
 * sentence*beam + d_parent[i*beam + s], in every self-attention key plane (one per block:
 * Section 3.2, shared layers keep no keys, so sharing shrinks this step too) and every
 * value plane; with self_is_aan it takes over the parent's running sum instead (when the
 * length is > 0).  d_parent holds beam slots 0..beam-1 of the SAME sentence, which is what
 * lets the gather run in place: all rows are read before any is written, as if copied
 * through a snapshot.  Slots with d_parent == s keep their rows and cost nothing.
 * Encoder memory is per sentence and is not touched.  max_len is a host bound on d_lens
 * (0 = capacity).  A parent outside 0..beam-1, a length outside 0..max_len or a sentence id
 * out of range skips that slot and is reported through san_device_status.  Bit copy. */
int32_t san_beam_reorder(san_ctx* ctx, const int32_t* d_sent_ids, const int32_t* d_parent,
                         const int32_t* d_lens, int32_t n_sent, int32_t max_len, void* stream);

/* Full-sequence shared attention (the encoder-side use of Table 5; with causal != 0 the
 * prefill of a decoder prompt): for every sequence i and head, the l x l weights
 *   S = Softmax(Q.K^T / sqrt(64)),  l = d_lens[i],  query row a over keys 0..l-1 (0..a when causal)
 * are computed once from the queries and keys of the block's lowest layer (Eq. 1, Eq. 3) and
 * applied to the values of each of the block's n_layers layers (Eq. 2, Eq. 4) in the same
 * launch.  Needs no context and allocates nothing.
 *   d_q, d_k  [n_seq][cap_len][n_heads][64]            (the order a projection writes them)
 *   d_v       [n_layers][n_seq][cap_len][n_heads][64]
 *   d_out     [n_layers][n_seq][cap_len][n_heads][64]  rows at or beyond d_lens[i] are not written
 *   d_S       optional [n_seq][n_heads][cap_len][ld_s] float32; entries a row does not attend
 *             to (causal) are written as 0, entries at or beyond d_lens[i] are not written
 * dtype must be SAN_BF16 (SAN_F32 is refused with SAN_ERR_UNSUPPORTED: tensor-core products
 * of float32 inputs would not meet the float32 tolerance).  max_len is a host bound on d_lens
 * (0 = cap_len); a longer length is cut to max_len.  It also selects the kernel: a bound of
 * 128 or more with n_layers <= 6 runs 128-query tiles on the tcgen05 tensor cores with the
 * accumulators in tensor memory (any length); otherwise 64-query tiles on mma.sync, for which
 * max_len above 512 is SAN_ERR_UNSUPPORTED. */
int32_t san_full_block(int32_t dtype, int32_t n_heads, int32_t n_layers, int32_t causal, const void* d_q,
                       const void* d_k, const void* d_v, const int32_t* d_lens, int32_t n_seq, int32_t cap_len,
                       int32_t max_len, float* d_S, int64_t ld_s, void* d_out, void* stream);

/* Policy learning (Section 3.1, Section 3.3, Eq. 6).
 *
 * san_js_matrix: the Jensen-Shannon divergence between the attention weights of every pair
 * of layers, JS(p,q) = (KL(p||m) + KL(q||m))/2 with m = (p+q)/2 and natural logarithms, one
 * value per (row, head) distribution and averaged over all of them (heads count as separate
 * channels).  d_S holds the weights of n_layers layers of an unshared model (block size 1) as
 * the decode step writes them: layer l at d_S + l*layer_stride, each [n_rows][n_heads][ld_s]
 * float32 with d_lens[row] valid positions (clamped to 0..ld_s).  d_js receives the
 * n_layers x n_layers symmetric matrix (float64, zero diagonal); it is cleared first.  Needs
 * no context and allocates nothing.
 *
 * san_block_similarity (host): Eq. 6 for the block of layers m..n (0-based, m < n),
 *   sim(m,n) = sum_{i != j in m..n} (ln 2 - JS(i,j)) / ((n-m+1)(n-m)).
 * san_policy_search (host): the bottom-up search of Section 3.3; starting at the lowest layer
 * a block grows while the similarity of the block with the next layer added is >= theta and
 * closes at the first failure (a block of one layer always qualifies); sizes[] (room for
 * n_layers entries) receives {pi_i}, ready for san_policy_set_sizes. js is a HOST matrix. */
int32_t san_js_matrix(int32_t n_layers, const float* d_S, int64_t layer_stride, int64_t ld_s,
                      int32_t n_rows, int32_t n_heads, const int32_t* d_lens, double* d_js, void* stream);
int32_t san_block_similarity(const double* js, int32_t n_layers, int32_t m, int32_t n, double* sim);
int32_t san_policy_search(const double* js, int32_t n_layers, double theta, int32_t* sizes, int32_t* n_blocks);

/* Reads (and clears) the device error word: *first_error = SAN_OK or the first
 * device-check error since the last read; detail[0..3] (optional) = kernel tag, item,
 * offending value, limit.  Synchronises `stream`. */
int32_t san_device_status(san_ctx* ctx, int32_t* first_error, int32_t* detail, void* stream);

/* The weights step of san_attn_weights for callers that cannot allocate device memory.
 * (The paper has no counterpart: this entry point exists for deployment reasons only.)
 *
 * A decode loop inside a serving process often may not call cudaMalloc: the server's
 * cache manager has reserved all of HBM, a plug-in contract forbids allocation while
 * serving, or the stall that cudaMalloc/cudaFree impose on every stream of the device is
 * not acceptable.  Such a caller cannot create a san_ctx, which needs a workspace buffer.
 * This call needs neither: it takes the key panel directly and keeps the scratch of
 * split rows (tickets, partial max/sum) in a fixed 1 MiB array inside the library image,
 * present on every GPU that loads the library until the process exits.  It calls no
 * cudaMalloc, cudaFree or other allocating routine.
 *
 *   dtype      SAN_F32 or SAN_BF16 (element type of d_q and d_K)
 *   n_queries  query rows sharing each key panel: 1 for self-attention, the beam size for
 *              encoder memory (1..8)
 *   d_q        [n_items][n_queries][n_heads][64]
 *   d_K        key plane [max_ids][n_heads][cap_len][64], the layout of the context's planes
 *   d_ids, d_lens, n_items, max_len, d_S, ld_s   as in san_attn_weights;
 *              d_S is [n_items][n_queries][n_heads][ld_s]
 *   d_status   optional device int32[8]: cleared, then [0] = SAN_ERR_DEVICE_CHECK and
 *              [1..4] = kernel tag, item, value, limit if an item was skipped
 *
 * Limits: n_items * n_heads <= 65536 rows, else SAN_ERR_CAPACITY (use a context instead).
 * The device that owns `stream` and every buffer must be the current device at the call, on
 * every call and not only the first (the call uses that device's copy of the array and does
 * not check whose stream it was given).  The first call on each device looks up the array's
 * device address; make that first call before any stream capture begins.  Every call on a
 * device uses the same array and finds what the previous call left there; the call clears
 * the tickets and status words it needs on `stream` before launching.  Two calls whose
 * kernels may overlap on one GPU (different streams without an event between them, or
 * different host threads doing so) race on the array: order them. */
int32_t san_attn_weights_static(int32_t dtype, int32_t n_heads, int32_t n_queries, const void* d_q,
                                const void* d_K, int32_t max_ids, int32_t cap_len,
                                const int32_t* d_ids, const int32_t* d_lens, int32_t n_items,
                                int32_t max_len, float* d_S, int64_t ld_s, int32_t* d_status,
                                void* stream);

const char* san_status_string(int32_t status);

#ifdef __cplusplus
}
#endif
#endif /* SAN_H_ */
