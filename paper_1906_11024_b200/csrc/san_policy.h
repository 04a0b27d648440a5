// Host-side sharing-policy tables (Section 3.3 of the paper): block sizes {pi_i} listed
// bottom-up, or a per-layer block id.  Pure integer work, no CUDA.
#pragma once

#include <stdint.h>

#include "../../include/san.h"

namespace san {

struct Policy {
    int32_t n_layers = 0;
    int32_t n_blocks = 0;
    int32_t block_of_layer[SAN_MAX_LAYERS];
    int32_t first_layer_of_block[SAN_MAX_LAYERS];
    int32_t size_of_block[SAN_MAX_LAYERS];

    bool is_first(int32_t layer) const { return first_layer_of_block[block_of_layer[layer]] == layer; }
};

// Both return SAN_OK or SAN_ERR_POLICY / SAN_ERR_NULL / SAN_ERR_SHAPE and leave *out
// untouched on error.
int32_t policy_from_sizes(const int32_t* sizes, int32_t n_blocks, int32_t n_layers, Policy* out);
int32_t policy_from_map(const int32_t* block_of_layer, int32_t n_layers, Policy* out);

// Eq. 6: similarity of the block of layers m..n (0-based, m < n) from the n_layers x n_layers
// matrix of pairwise JS divergences, with mu(i, j) = ln 2 - JS(i, j).
double block_similarity(const double* js, int32_t n_layers, int32_t m, int32_t n);
// Section 3.3 search: bottom-up, each block grows while the similarity of the block with the
// next layer added stays >= theta.  Writes the block sizes; returns their number.
int32_t search_policy(const double* js, int32_t n_layers, double theta, int32_t* sizes);

}  // namespace san
