// Policy learning, device part (Section 3.1 and 3.3): the Jensen-Shannon divergence between
// the attention weights of every pair of layers,
//     JS(p, q) = (KL(p || m) + KL(q || m)) / 2,   m = (p + q) / 2,   0 ln 0 = 0,
// one value per (row, head) distribution, averaged over rows and heads (heads are separate
// channels).  Input is the weights of an unshared model as the decode step writes them:
// S [layer][row][head][ld] float32 with lens[row] valid positions per row.
//
// One warp per (row, head): for every pair of layers the lanes stride over the positions,
// the warp reduces, lane 0 adds the pair's value to a double accumulator.  The weights of a
// row (layers x len floats, a few KB) are read from L1/L2 after the first pair; the whole
// input is read from HBM once.  Logarithms are __logf on float32 weights; the sum over
// positions is float32 per lane, the sum over rows double.
#pragma once

#include "san_kernels.cuh"

namespace san {

struct JsParams {
    const float* S; long long layer_stride, ld;     // floats between layers / between (row, head) distributions
    const int* lens;
    int n_layers, n_rows, n_heads;
    double* js;                                     // [n_layers][n_layers], sums until js_finish_kernel
};

static __global__ void __launch_bounds__(256) js_pairs_kernel(const JsParams p) {
    const int lane = threadIdx.x & 31;
    const long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (w >= (long long)p.n_rows * p.n_heads) return;
    const int row = (int)(w / p.n_heads);
    int len = p.lens[row];
    len = len < 0 ? 0 : (len > p.ld ? (int)p.ld : len);
    const float* base = p.S + w * p.ld;
    for (int a = 0; a < p.n_layers; ++a) {
        const float* Sa = base + (long long)a * p.layer_stride;
        for (int b = a + 1; b < p.n_layers; ++b) {
            const float* Sb = base + (long long)b * p.layer_stride;
            float acc = 0.f;
            for (int j = lane; j < len; j += 32) {
                const float x = Sa[j], y = Sb[j], m = 0.5f * (x + y);
                // x / m lies in (0, 2]: the fast logarithm is within 2^-21 absolute there (2 ulp below
                // 1/2), so a row's value, a sum of terms weighted by x with sum(x) = 1, stays within 3e-7
                if (x > 0.f) acc += 0.5f * x * __logf(__fdividef(x, m));
                if (y > 0.f) acc += 0.5f * y * __logf(__fdividef(y, m));
            }
            acc = warp_sum(acc);
            if (lane == 0) atomicAdd(p.js + (long long)a * p.n_layers + b, (double)acc);
        }
    }
}

// Sums above the diagonal -> means, mirrored; zero diagonal.
static __global__ void js_finish_kernel(double* js, int n_layers, double count) {
    const int a = blockIdx.x, b = threadIdx.x;
    if (a >= n_layers || b >= n_layers) return;
    if (a < b) {
        const double v = count > 0.0 ? js[(long long)a * n_layers + b] / count : 0.0;
        js[(long long)a * n_layers + b] = v;
        js[(long long)b * n_layers + a] = v;
    } else if (a == b) {
        js[(long long)a * n_layers + a] = 0.0;
    }
}

}  // namespace san
