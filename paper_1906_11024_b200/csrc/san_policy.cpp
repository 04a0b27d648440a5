#include "san_policy.h"

#include <cmath>

namespace san {

int32_t policy_from_sizes(const int32_t* sizes, int32_t n_blocks, int32_t n_layers, Policy* out) {
    if (!sizes || !out) return SAN_ERR_NULL;
    if (n_layers < 1 || n_layers > SAN_MAX_LAYERS) return SAN_ERR_SHAPE;
    if (n_blocks < 1 || n_blocks > n_layers) return SAN_ERR_POLICY;
    Policy p;
    p.n_layers = n_layers;
    p.n_blocks = n_blocks;
    int64_t next = 0;   // lowest layer of the block being laid out
    for (int32_t b = 0; b < n_blocks; ++b) {
        const int32_t pi = sizes[b];
        if (pi < 1 || next + pi > n_layers) return SAN_ERR_POLICY;
        p.first_layer_of_block[b] = (int32_t)next;
        p.size_of_block[b] = pi;
        for (int32_t k = 0; k < pi; ++k) p.block_of_layer[next + k] = b;
        next += pi;
    }
    if (next != n_layers) return SAN_ERR_POLICY;   // the sizes must add up to the stack height
    *out = p;
    return SAN_OK;
}

int32_t policy_from_map(const int32_t* block_of_layer, int32_t n_layers, Policy* out) {
    if (!block_of_layer || !out) return SAN_ERR_NULL;
    if (n_layers < 1 || n_layers > SAN_MAX_LAYERS) return SAN_ERR_SHAPE;
    Policy p;
    p.n_layers = n_layers;
    p.n_blocks = 0;
    for (int32_t layer = 0; layer < n_layers; ++layer) {
        const int32_t id = block_of_layer[layer];
        if (id == p.n_blocks - 1 && layer > 0) {           // same block as the layer below
            p.size_of_block[id] += 1;
        } else if (id == p.n_blocks) {                     // a new block opens here
            p.first_layer_of_block[id] = layer;
            p.size_of_block[id] = 1;
            p.n_blocks += 1;
        } else {
            return SAN_ERR_POLICY;                         // ids skip, fall, or do not start at 0
        }
        p.block_of_layer[layer] = id;
    }
    *out = p;
    return SAN_OK;
}

double block_similarity(const double* js, int32_t n_layers, int32_t m, int32_t n) {
    const double ln2 = std::log(2.0);
    double mu = 0.0;
    for (int32_t i = m; i <= n; ++i)
        for (int32_t j = m; j <= n; ++j)
            if (i != j) mu += ln2 - js[(int64_t)i * n_layers + j];
    const double layers = (double)(n - m + 1);
    return mu / (layers * (layers - 1.0));           // ordered pairs i != j inside the block
}

int32_t search_policy(const double* js, int32_t n_layers, double theta, int32_t* sizes) {
    int32_t n_blocks = 0;
    for (int32_t m = 0; m < n_layers;) {
        int32_t top = m;                               // a block of one layer always qualifies
        while (top + 1 < n_layers && block_similarity(js, n_layers, m, top + 1) >= theta) ++top;
        sizes[n_blocks++] = top - m + 1;
        m = top + 1;
    }
    return n_blocks;
}

}  // namespace san
