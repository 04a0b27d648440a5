/*
 * CPU oracle for shared-attention (SAN) decoding.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow restatement of what the paper defines, used to check the CUDA
 * library and as the timed CPU baseline.  It shares no code, header, layout or
 * table with the CUDA path.  Inputs are float (already rounded to the storage
 * dtype by the input generator); every sum, product, exponential and division
 * is done in double.
 *
 * What is computed (notation of the paper: S = weights, A = S.V = output; the
 * output is called O here to keep it apart from the weights):
 *
 *   Eq. 1   S = Softmax(q.K^T / sqrt(d_k)), one query row per (sequence, head)
 *           in cached decoding; the softmax runs over the cached positions.
 *           d_k is the per-head width d_h (Section 4.1 gives the model width
 *           512 with 8 heads).
 *   Eq. 2   O = S.V
 *   Eq. 3-4 in a block of pi adjacent layers only the lowest layer m computes
 *           S^m = s(Q^m, K^m); layers m+1 .. m+pi-1 reuse S^m and apply it to
 *           their own V.
 *   Eq. 5   encoder-decoder attention with shared context: A^{m+i} = A^m.
 *           (Table 4 also lists the variant where each layer keeps its own V;
 *           both are available, chosen by `encdec_shared_context`.)
 *   AAN     the average-attention model the paper pairs with SAN (Table 6):
 *           the output at target position t is the mean of the inputs at
 *           positions 1..t (the paper cites it without a formula; this is the
 *           cumulative average of that model).
 *   Eq. 6   sim(m,n) over a block, with mu(i,j) = ln 2 - JS(i,j), and the
 *           bottom-up block search of Section 3.3.
 *
 * Own storage layout: [layer][seq][pos][head][dim] (position-major), which is
 * deliberately not the layout the CUDA library uses.
 *
 * Pins (tests/test_oracle_*.py): textbook multi-head attention through a
 * library routine for block size 1, rows of S summing to one, S_first.V_layer
 * recomputed with a separate matrix product, closed forms (length 1, uniform
 * weights = prefix mean = AAN, shift and permutation invariance, one-hot
 * limit), a hand-worked example, brute force over every policy of tiny
 * stacks, and the Figure 2 matrices for Eq. 6.  No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_ERR_POLICY 3
#define ORC_ERR_RANGE 6

typedef struct oracle_san {
    int M, H, dh, n_seqs, beam, n_sent, max_tgt, max_src;
    int n_self, n_enc;
    int *self_block, *self_first; /* [M], [n_self] */
    int *enc_block, *enc_first;   /* [M], [n_enc]  */
    int encdec_shared_context;    /* Eq. 5 on/off */
    float **Kself, **Vself;       /* per layer: [n_seqs][max_tgt][H][dh] */
    float **Kmem, **Vmem;         /* per layer: [n_sent][max_src][H][dh] */
    int *src_len;                 /* [n_sent] */
    double **S_self;              /* per self block: [n_seqs][H][max_tgt] */
    double **S_enc;               /* per enc-dec block: [n_seqs][H][max_src] */
    double **O_enc;               /* per enc-dec block: [n_seqs][H][dh] (Eq. 5) */
    float **Xaan;                 /* per layer: [n_seqs][max_tgt][H*dh] */
} oracle_san;

/* ------------------------------------------------------------------ policy */

/* Sharing policy {pi_1..pi_N} listed bottom-up (Section 3.3): sizes must be
 * >= 1 and sum to M.  Writes layer -> block and block -> lowest layer. */
int oracle_policy_from_sizes(const int *sizes, int n_blocks, int M,
                             int *block_of_layer, int *first_layer_of_block) {
    if (!sizes || n_blocks < 1 || M < 1) return ORC_ERR_POLICY;
    int layer = 0;
    for (int b = 0; b < n_blocks; ++b) {
        if (sizes[b] < 1) return ORC_ERR_POLICY;
        if (layer + sizes[b] > M) return ORC_ERR_POLICY;
        first_layer_of_block[b] = layer;
        for (int i = 0; i < sizes[b]; ++i) block_of_layer[layer++] = b;
    }
    return layer == M ? ORC_OK : ORC_ERR_POLICY;
}

/* The same policy given as a per-layer block id: ids start at 0 and each next
 * layer keeps the id or raises it by one (blocks are runs of adjacent layers). */
int oracle_policy_from_map(const int *block_of_layer, int M, int *sizes,
                           int *first_layer_of_block, int *n_blocks) {
    if (!block_of_layer || M < 1 || block_of_layer[0] != 0) return ORC_ERR_POLICY;
    int nb = 0;
    for (int l = 0; l < M; ++l) {
        int prev = l ? block_of_layer[l - 1] : -1;
        if (block_of_layer[l] == prev) {
            sizes[nb - 1] += 1;
        } else if (block_of_layer[l] == prev + 1) {
            first_layer_of_block[nb] = l;
            sizes[nb] = 1;
            ++nb;
        } else {
            return ORC_ERR_POLICY;
        }
    }
    *n_blocks = nb;
    return ORC_OK;
}

/* --------------------------------------------------------------- lifetime */

static void *zalloc(size_t n, size_t sz) { return calloc(n ? n : 1, sz); }

oracle_san *oracle_create(int M, int H, int dh, int n_sent, int beam, int max_tgt, int max_src,
                          const int *self_sizes, int n_self, const int *enc_sizes, int n_enc,
                          int encdec_shared_context) {
    oracle_san *o = (oracle_san *)zalloc(1, sizeof(*o));
    o->M = M; o->H = H; o->dh = dh; o->n_sent = n_sent; o->beam = beam;
    o->n_seqs = n_sent * beam; o->max_tgt = max_tgt; o->max_src = max_src;
    o->n_self = n_self; o->n_enc = n_enc; o->encdec_shared_context = encdec_shared_context;
    o->self_block = (int *)zalloc(M, sizeof(int)); o->self_first = (int *)zalloc(n_self, sizeof(int));
    o->enc_block = (int *)zalloc(M, sizeof(int)); o->enc_first = (int *)zalloc(n_enc, sizeof(int));
    if (oracle_policy_from_sizes(self_sizes, n_self, M, o->self_block, o->self_first) != ORC_OK ||
        oracle_policy_from_sizes(enc_sizes, n_enc, M, o->enc_block, o->enc_first) != ORC_OK) {
        free(o->self_block); free(o->self_first); free(o->enc_block); free(o->enc_first); free(o);
        return NULL;
    }
    size_t self_elems = (size_t)o->n_seqs * max_tgt * H * dh;
    size_t mem_elems = (size_t)n_sent * max_src * H * dh;
    o->Kself = (float **)zalloc(M, sizeof(float *)); o->Vself = (float **)zalloc(M, sizeof(float *));
    o->Kmem = (float **)zalloc(M, sizeof(float *)); o->Vmem = (float **)zalloc(M, sizeof(float *));
    o->Xaan = (float **)zalloc(M, sizeof(float *));
    for (int l = 0; l < M; ++l) {   /* calloc pages stay untouched until written */
        o->Kself[l] = (float *)zalloc(self_elems, sizeof(float));
        o->Vself[l] = (float *)zalloc(self_elems, sizeof(float));
        o->Xaan[l] = (float *)zalloc(self_elems, sizeof(float));
        o->Kmem[l] = (float *)zalloc(mem_elems, sizeof(float));
        o->Vmem[l] = (float *)zalloc(mem_elems, sizeof(float));
    }
    o->src_len = (int *)zalloc(n_sent, sizeof(int));
    o->S_self = (double **)zalloc(n_self, sizeof(double *));
    for (int b = 0; b < n_self; ++b) o->S_self[b] = (double *)zalloc((size_t)o->n_seqs * H * max_tgt, sizeof(double));
    o->S_enc = (double **)zalloc(n_enc, sizeof(double *));
    o->O_enc = (double **)zalloc(n_enc, sizeof(double *));
    for (int b = 0; b < n_enc; ++b) {
        o->S_enc[b] = (double *)zalloc((size_t)o->n_seqs * H * max_src, sizeof(double));
        o->O_enc[b] = (double *)zalloc((size_t)o->n_seqs * H * dh, sizeof(double));
    }
    return o;
}

void oracle_destroy(oracle_san *o) {
    if (!o) return;
    for (int l = 0; l < o->M; ++l) {
        free(o->Kself[l]); free(o->Vself[l]); free(o->Xaan[l]); free(o->Kmem[l]); free(o->Vmem[l]);
    }
    for (int b = 0; b < o->n_self; ++b) free(o->S_self[b]);
    for (int b = 0; b < o->n_enc; ++b) { free(o->S_enc[b]); free(o->O_enc[b]); }
    free(o->Kself); free(o->Vself); free(o->Xaan); free(o->Kmem); free(o->Vmem);
    free(o->S_self); free(o->S_enc); free(o->O_enc); free(o->src_len);
    free(o->self_block); free(o->self_first); free(o->enc_block); free(o->enc_first);
    free(o);
}

/* ------------------------------------------------------------------ caches */

/* Attention cache (Section 4.1): keep this step's key and value rows of every
 * listed sequence at position pos[i].  k may be NULL (a layer that reuses
 * another layer's weights has no keys).  k, v: [n][H][dh]. */
int oracle_self_append(oracle_san *o, int layer, int n, const int *seq_ids, const int *pos,
                       const float *k, const float *v) {
    if (layer < 0 || layer >= o->M) return ORC_ERR_RANGE;
    size_t row = (size_t)o->H * o->dh;
    for (int i = 0; i < n; ++i) {
        int s = seq_ids[i], p = pos[i];
        if (s < 0 || s >= o->n_seqs || p < 0 || p >= o->max_tgt) return ORC_ERR_RANGE;
        size_t at = ((size_t)s * o->max_tgt + p) * row;
        if (k) memcpy(o->Kself[layer] + at, k + (size_t)i * row, row * sizeof(float));
        if (v) memcpy(o->Vself[layer] + at, v + (size_t)i * row, row * sizeof(float));
    }
    return ORC_OK;
}

/* Encoder memory of one sentence for one layer (keys and values come from the
 * encoder output, Section 2): Ls rows of [H][dh], consecutive rows row_stride
 * floats apart.  K may be NULL. */
int oracle_mem_set(oracle_san *o, int layer, int sentence, int Ls, const float *K, const float *V,
                   long row_stride) {
    if (layer < 0 || layer >= o->M || sentence < 0 || sentence >= o->n_sent || Ls < 1 || Ls > o->max_src)
        return ORC_ERR_RANGE;
    size_t row = (size_t)o->H * o->dh;
    o->src_len[sentence] = Ls;
    for (int j = 0; j < Ls; ++j) {
        size_t at = ((size_t)sentence * o->max_src + j) * row;
        if (K) memcpy(o->Kmem[layer] + at, K + (size_t)j * row_stride, row * sizeof(float));
        if (V) memcpy(o->Vmem[layer] + at, V + (size_t)j * row_stride, row * sizeof(float));
    }
    return ORC_OK;
}

/* Beam search keeps, for every surviving hypothesis, the cache of the parent
 * it extends (Section 4.1 decodes with beam 4): sequence s takes over the
 * first len[s] cached rows (keys, values, AAN inputs) of sequence src[s], for
 * every layer.  All reads happen before any write. */
int oracle_beam_reorder(oracle_san *o, const int *src, const int *len) {
    size_t row = (size_t)o->H * o->dh;
    size_t per_seq = (size_t)o->max_tgt * row;
    for (int s = 0; s < o->n_seqs; ++s)
        if (src[s] < 0 || src[s] >= o->n_seqs || len[s] < 0 || len[s] > o->max_tgt) return ORC_ERR_RANGE;
    float *tmp = (float *)zalloc((size_t)o->n_seqs * per_seq, sizeof(float));
    for (int l = 0; l < o->M; ++l) {
        float *planes[3] = {o->Kself[l], o->Vself[l], o->Xaan[l]};
        for (int a = 0; a < 3; ++a) {
            memcpy(tmp, planes[a], (size_t)o->n_seqs * per_seq * sizeof(float));
            for (int s = 0; s < o->n_seqs; ++s)
                memcpy(planes[a] + (size_t)s * per_seq, tmp + (size_t)src[s] * per_seq,
                       (size_t)len[s] * row * sizeof(float));
        }
    }
    free(tmp);
    return ORC_OK;
}

/* --------------------------------------------------------------- attention */

/* Eq. 1 for one query row: z_j = (q . K_j) / sqrt(dh), S = exp(z - max z) / sum.
 * Subtracting the maximum does not change the quotient; it keeps exp in range.
 * K_j sits at Krows + j*stride. */
static void weights_row(const float *q, const float *Krows, size_t stride, int len, int dh, double *S) {
    double scale = 1.0 / sqrt((double)dh);
    double zmax = -INFINITY;
    for (int j = 0; j < len; ++j) {
        double dot = 0.0;
        for (int d = 0; d < dh; ++d) dot += (double)q[d] * (double)Krows[(size_t)j * stride + d];
        S[j] = dot * scale;
        if (S[j] > zmax) zmax = S[j];
    }
    double sum = 0.0;
    for (int j = 0; j < len; ++j) { S[j] = exp(S[j] - zmax); sum += S[j]; }
    for (int j = 0; j < len; ++j) S[j] /= sum;
}

/* Eq. 2 for one query row: O_d = sum_j S_j V_{j,d}. */
static void apply_row(const double *S, const float *Vrows, size_t stride, int len, int dh, double *O) {
    for (int d = 0; d < dh; ++d) {
        double acc = 0.0;
        for (int j = 0; j < len; ++j) acc += S[j] * (double)Vrows[(size_t)j * stride + d];
        O[d] = acc;
    }
}

/* Decoder self-attention of one layer for the listed sequences over the first
 * lens[i] cached positions.  If the layer is the lowest of its block it
 * computes and keeps S from q (Eq. 3); otherwise it reuses the block's S
 * (Eq. 4) and q is not read (may be NULL).  Every layer then applies S to its
 * own cached values (Eq. 2).
 *   q      [n][H][dh] float
 *   S_out  [n][H][ld_s] double or NULL (the weights this layer used)
 *   O_out  [n][H][dh] double */
int oracle_self_attend(oracle_san *o, int layer, int n, const int *seq_ids, const int *lens,
                       const float *q, double *S_out, long ld_s, double *O_out) {
    if (layer < 0 || layer >= o->M) return ORC_ERR_RANGE;
    int H = o->H, dh = o->dh, b = o->self_block[layer];
    int is_first = (o->self_first[b] == layer);
    if (is_first && !q) return ORC_ERR_RANGE;
    for (int i = 0; i < n; ++i)
        if (seq_ids[i] < 0 || seq_ids[i] >= o->n_seqs || lens[i] < 1 || lens[i] > o->max_tgt) return ORC_ERR_RANGE;
    size_t stride = (size_t)H * dh;
#pragma omp parallel for collapse(2) schedule(dynamic, 4)
    for (int i = 0; i < n; ++i) {
        for (int h = 0; h < H; ++h) {
            int s = seq_ids[i], len = lens[i];
            double *S = o->S_self[b] + ((size_t)s * H + h) * o->max_tgt;
            size_t base = (size_t)s * o->max_tgt * stride + (size_t)h * dh;
            if (is_first)
                weights_row(q + ((size_t)i * H + h) * dh, o->Kself[layer] + base, stride, len, dh, S);
            apply_row(S, o->Vself[layer] + base, stride, len, dh, O_out + ((size_t)i * H + h) * dh);
            if (S_out) memcpy(S_out + ((size_t)i * H + h) * ld_s, S, (size_t)len * sizeof(double));
        }
    }
    return ORC_OK;
}

/* Encoder-decoder attention of one layer: the same two equations over the
 * encoder memory of the sequence's sentence (sentence = seq / beam; the beams
 * of a sentence read the same memory).  With shared context (Eq. 5) a layer
 * that is not the lowest of its block returns the block's stored output. */
int oracle_encdec_attend(oracle_san *o, int layer, int n, const int *seq_ids, const float *q,
                         double *S_out, long ld_s, double *O_out) {
    if (layer < 0 || layer >= o->M) return ORC_ERR_RANGE;
    int H = o->H, dh = o->dh, b = o->enc_block[layer];
    int is_first = (o->enc_first[b] == layer);
    if (is_first && !q) return ORC_ERR_RANGE;
    for (int i = 0; i < n; ++i) {
        if (seq_ids[i] < 0 || seq_ids[i] >= o->n_seqs) return ORC_ERR_RANGE;
        if (o->src_len[seq_ids[i] / o->beam] < 1) return ORC_ERR_RANGE;
    }
    size_t stride = (size_t)H * dh;
#pragma omp parallel for collapse(2) schedule(dynamic, 4)
    for (int i = 0; i < n; ++i) {
        for (int h = 0; h < H; ++h) {
            int s = seq_ids[i], sent = s / o->beam, len = o->src_len[sent];
            double *S = o->S_enc[b] + ((size_t)s * H + h) * o->max_src;
            double *Ob = o->O_enc[b] + ((size_t)s * H + h) * dh;
            double *Oi = O_out + ((size_t)i * H + h) * dh;
            size_t base = (size_t)sent * o->max_src * stride + (size_t)h * dh;
            if (is_first)
                weights_row(q + ((size_t)i * H + h) * dh, o->Kmem[layer] + base, stride, len, dh, S);
            if (o->encdec_shared_context) {
                if (is_first) apply_row(S, o->Vmem[layer] + base, stride, len, dh, Ob);
                memcpy(Oi, Ob, (size_t)dh * sizeof(double));
            } else {
                apply_row(S, o->Vmem[layer] + base, stride, len, dh, Oi);
            }
            if (S_out) memcpy(S_out + ((size_t)i * H + h) * ld_s, S, (size_t)len * sizeof(double));
        }
    }
    return ORC_OK;
}

/* Average attention in place of decoder self-attention: keep x at position
 * t[i] (1-based) and return the mean of positions 1..t[i].  The history is
 * summed afresh every call: the definition, not a running recurrence.
 *   x [n][H*dh] float, out [n][H*dh] double */
int oracle_aan_step(oracle_san *o, int layer, int n, const int *seq_ids, const int *t,
                    const float *x, double *out) {
    if (layer < 0 || layer >= o->M) return ORC_ERR_RANGE;
    size_t d = (size_t)o->H * o->dh;
    for (int i = 0; i < n; ++i)
        if (seq_ids[i] < 0 || seq_ids[i] >= o->n_seqs || t[i] < 1 || t[i] > o->max_tgt) return ORC_ERR_RANGE;
#pragma omp parallel for schedule(dynamic, 4)
    for (int i = 0; i < n; ++i) {
        float *hist = o->Xaan[layer] + (size_t)seq_ids[i] * o->max_tgt * d;
        memcpy(hist + (size_t)(t[i] - 1) * d, x + (size_t)i * d, d * sizeof(float));
        for (size_t c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int k = 0; k < t[i]; ++k) acc += (double)hist[(size_t)k * d + c];
            out[(size_t)i * d + c] = acc / (double)t[i];
        }
    }
    return ORC_OK;
}

/* Full-sequence SAN (the encoder-side use of Table 5): one l x l weight matrix
 * per head computed by the lowest layer of a block (Eq. 1 with l query rows)
 * and applied to each layer's own V (Eq. 2).  causal != 0 restricts query i to
 * keys 0..i (decoder prefill).  Q,K: [l][H][dh]; V: [n_layers][l][H][dh];
 * S_out: [H][l][l] (or NULL); O_out: [n_layers][l][H][dh]. */
int oracle_full_block(int l, int H, int dh, int n_layers, int causal, const float *Q, const float *K,
                      const float *V, double *S_out, double *O_out) {
    if (l < 1 || H < 1 || dh < 1 || n_layers < 1) return ORC_ERR_RANGE;
    size_t stride = (size_t)H * dh;
#pragma omp parallel for collapse(2) schedule(dynamic, 4)
    for (int h = 0; h < H; ++h) {
        for (int i = 0; i < l; ++i) {
            double *S = (double *)malloc((size_t)l * sizeof(double));
            int len = causal ? i + 1 : l;
            weights_row(Q + (size_t)i * stride + (size_t)h * dh, K + (size_t)h * dh, stride, len, dh, S);
            for (int j = len; j < l; ++j) S[j] = 0.0;
            if (S_out) memcpy(S_out + ((size_t)h * l + i) * l, S, (size_t)l * sizeof(double));
            for (int a = 0; a < n_layers; ++a)
                apply_row(S, V + (size_t)a * l * stride + (size_t)h * dh, stride, len, dh,
                          O_out + ((size_t)a * l + i) * stride + (size_t)h * dh);
            free(S);
        }
    }
    return ORC_OK;
}

/* ---------------------------------------------------------- policy learner */

/* Jensen-Shannon divergence (natural log) of two distributions over n points:
 * JS = (KL(p||m) + KL(q||m)) / 2 with m = (p+q)/2, and 0 ln 0 = 0.  It is
 * symmetric and bounded by ln 2 (Section 3.1). */
double oracle_js_divergence(const double *p, const double *q, int n) {
    double js = 0.0;
    for (int i = 0; i < n; ++i) {
        double m = 0.5 * (p[i] + q[i]);
        if (p[i] > 0.0) js += 0.5 * p[i] * log(p[i] / m);
        if (q[i] > 0.0) js += 0.5 * q[i] * log(q[i] / m);
    }
    return js;
}

/* JS between two layers' weights: one score per (row, head) distribution,
 * then averaged (heads are separate channels, Section 3.1).  Sa, Sb:
 * [n_rows][H][ld] with row i holding lens[i] probabilities per head. */
double oracle_layer_js(const double *Sa, const double *Sb, int n_rows, int H, long ld, const int *lens) {
    double acc = 0.0;
    for (int i = 0; i < n_rows; ++i)
        for (int h = 0; h < H; ++h)
            acc += oracle_js_divergence(Sa + ((size_t)i * H + h) * ld, Sb + ((size_t)i * H + h) * ld, lens[i]);
    return acc / ((double)n_rows * H);
}

/* Eq. 6: similarity of block b(m,n) (1-based layers, m < n) from the M x M
 * matrix of pairwise JS divergences, with mu(i,j) = ln 2 - JS(i,j). */
double oracle_block_sim(const double *JS, int M, int m, int n) {
    double acc = 0.0;
    for (int i = m; i <= n; ++i)
        for (int j = m; j <= n; ++j)
            if (i != j) acc += log(2.0) - JS[(size_t)(i - 1) * M + (j - 1)];
    return acc / ((double)(n - m + 1) * (double)(n - m));
}

/* Section 3.3 search: start at layer 1, grow the block upward while
 * sim(m, n+1) >= theta, close it at the first failure, continue from the next
 * layer.  A block of one layer always qualifies (Eq. 6 is undefined there).
 * Writes the block sizes bottom-up; returns the number of blocks. */
int oracle_greedy_policy(const double *JS, int M, double theta, int *sizes) {
    int nb = 0, m = 1;
    while (m <= M) {
        int n = m;
        while (n + 1 <= M && oracle_block_sim(JS, M, m, n + 1) >= theta) ++n;
        sizes[nb++] = n - m + 1;
        m = n + 1;
    }
    return nb;
}
