// Microbenchmark: how fast the GPU can read the self-attention access pattern of the sentence-sized
// workload at all: 9 planes x 2048 (sequence, head) panels of 6..33 rows of 128 bytes, panels
// 66 rows apart, one warp per panel with plain 16-byte loads, launches rotating over six copies
// of the arena.  The best time is what a kernel that did nothing but read these bytes would need,
// launch and ramp included.
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -o panel_read_floor panel_read_floor.cu && ./panel_read_floor
#include <cstdio>
#include <cstdlib>
#include <cstdint>
#include <cuda_runtime.h>
#include <vector>
__global__ void rd(const uint4* base, const int* lens, int n_panels, int planes, size_t plane_stride16, int cap, unsigned* sink) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int total = n_panels * planes;
    unsigned acc = 0;
    for (int w = warp; w < total; w += (gridDim.x * blockDim.x) >> 5) {
        const int pl = w / n_panels, pn = w % n_panels;
        const int L = lens[pn >> 3];
        const uint4* p = base + pl * plane_stride16 + (size_t)pn * cap * 8;
        for (int i = lane; i < L * 8; i += 32) { uint4 v = __ldg(p + i); acc += v.x ^ v.y ^ v.z ^ v.w; }
    }
    if (acc == 0x12345678u) sink[0] = acc;
}
int main(int argc, char** argv) {
    // optional arguments: rows a panel has room for (default 66), rows read of every panel (default 0: 6..33, as the workload)
    const int cap = argc > 1 ? atoi(argv[1]) : 66, fixed = argc > 2 ? atoi(argv[2]) : 0;
    const int seqs = 256, H = 8, planes = 9, R = 6;
    const int n_panels = seqs * H;
    const size_t plane_bytes = (size_t)n_panels * cap * 128;
    const size_t rep_bytes = plane_bytes * 16;      // a replica also holds other planes between
    char* buf; cudaMalloc(&buf, rep_bytes * R); cudaMemset(buf, 1, rep_bytes * R);
    std::vector<int> lens(seqs);
    size_t bytes = 0;
    for (int s = 0; s < seqs; ++s) { lens[s] = fixed > 0 ? fixed : 6 + ((s / 4) * 7919) % 28; bytes += (size_t)lens[s] * 128 * H * planes; }
    int* dl; cudaMalloc(&dl, seqs * 4); cudaMemcpy(dl, lens.data(), seqs * 4, cudaMemcpyHostToDevice);
    unsigned* sink; cudaMalloc(&sink, 4);
    cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
    for (int blocks : {148, 296, 592, 1184, 2368}) for (int threads : {256, 512, 1024}) {
        for (int it = 0; it < 3; ++it) rd<<<blocks, threads>>>((const uint4*)(buf + (it % R) * rep_bytes), dl, n_panels, planes, plane_bytes / 16, cap, sink);
        cudaEventRecord(e0);
        const int iters = 60;
        for (int it = 0; it < iters; ++it) rd<<<blocks, threads>>>((const uint4*)(buf + (it % R) * rep_bytes), dl, n_panels, planes, plane_bytes / 16, cap, sink);
        cudaEventRecord(e1); cudaEventSynchronize(e1);
        float ms; cudaEventElapsedTime(&ms, e0, e1);
        printf("blocks %4d threads %4d: %.2f us per pass, %.0f GB/s (%.1f MB)\n", blocks, threads, ms * 1e3 / iters, bytes / (ms * 1e-3 / iters) / 1e9, bytes / 1e6);
    }
    return 0;
}
