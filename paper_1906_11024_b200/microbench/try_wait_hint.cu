// Microbenchmark: how long one mbarrier.try_wait holds the thread when the phase does not complete,
// without and with a suspend-time hint.  The barrier is never completed here; the loops are
// counted, not conditional, so the kernel always ends.
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -o try_wait_hint try_wait_hint.cu && ./try_wait_hint
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
__global__ void k(long long* out) {
    __shared__ uint64_t bar;
    uint32_t b = (uint32_t)__cvta_generic_to_shared(&bar);
    if (threadIdx.x == 0) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(b), "r"(1));
    __syncthreads();
    uint32_t ok;
    long long t0 = clock64();
    for (int i = 0; i < 8; ++i)
        asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(ok) : "r"(b), "r"(0) : "memory");
    long long t1 = clock64();
    for (int i = 0; i < 8; ++i)
        asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(ok) : "r"(b), "r"(0), "r"(20000) : "memory");
    long long t2 = clock64();
    for (int i = 0; i < 8; ++i)
        asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(ok) : "r"(b), "r"(0), "r"(1000000) : "memory");
    long long t3 = clock64();
    if (threadIdx.x == 0) { out[0] = (t1 - t0) / 8; out[1] = (t2 - t1) / 8; out[2] = (t3 - t2) / 8; out[3] = ok; }
}
int main() {
    long long* out; cudaMallocManaged(&out, 64);
    k<<<1, 32>>>(out);
    if (cudaDeviceSynchronize() != cudaSuccess) { printf("error\n"); return 1; }
    printf("try_wait blocks: no hint %lld cycles, hint 20000 %lld cycles, hint 1000000 %lld cycles\n", out[0], out[1], out[2]);
    return 0;
}
