// Microbenchmark behind the step kernels' copy design: how many cycles a warp spends issuing
// cp.async.bulk copies (global -> shared, completion on an mbarrier), as a function of the copy
// size, of the lanes that issue in one instruction and of the warps that issue at once, and how
// long until the data has landed.  Every access is in bounds and every wait is bounded.
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -o bulk_copy_issue bulk_copy_issue.cu && ./bulk_copy_issue
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
__device__ __forceinline__ uint32_t s32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool try_wait(uint32_t bar, uint32_t par) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(ok) : "r"(bar), "r"(par) : "memory");
    return ok;
}
extern __shared__ __align__(128) unsigned char sm[];
__global__ void k(const char* src, size_t src_bytes, int bytes, int lanes, int warps, int rounds, long long* out) {
    __shared__ uint64_t bars[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x < 32) { asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(&bars[threadIdx.x])), "r"(1)); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    if (warp >= warps) return;
    const uint32_t bar = s32(&bars[warp]);
    const uint32_t dst0 = s32(sm) + warp * (lanes * bytes);
    long long issue = 0, total = 0;
    uint32_t par = 0;
    size_t at = ((size_t)blockIdx.x * 32 + warp) * 1048576 % src_bytes;
    for (int r = 0; r < rounds; ++r) {
        const long long t0 = clock64();
        if (lane == 0) asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(lanes * bytes) : "memory");
        if (lane < lanes) {
            const char* s = src + (at + (size_t)lane * 65536) % (src_bytes - 65536);
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst0 + lane * bytes), "l"(s), "r"(bytes), "r"(bar) : "memory");
        }
        __syncwarp();
        const long long t1 = clock64();
        long long spin = 0;
        while (!try_wait(bar, par) && spin < 100000000) ++spin;
        par ^= 1;
        const long long t2 = clock64();
        issue += t1 - t0; total += t2 - t0;
        at = (at + 7340032) % src_bytes;
    }
    if (lane == 0 && blockIdx.x == 0) { out[warp * 2] = issue / rounds; out[warp * 2 + 1] = total / rounds; }
}
int main() {
    const size_t SB = 1ull << 30;
    char* src; cudaMalloc(&src, SB); cudaMemset(src, 1, SB);
    long long* out; cudaMallocManaged(&out, 64 * 8);
    cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    int sizes[] = {128, 1024, 2432, 4096};
    for (int bytes : sizes) for (int lanes : {1, 8, 24}) for (int warps : {1, 4, 16}) {
        if ((size_t)warps * lanes * bytes > 200 * 1024) continue;
        for (int i = 0; i < 64; ++i) out[i] = 0;
        k<<<148, 512, 200 * 1024>>>(src, SB, bytes, lanes, warps, 50, out);
        cudaError_t e = cudaDeviceSynchronize();
        if (e != cudaSuccess) { printf("error %s\n", cudaGetErrorString(e)); return 1; }
        printf("bytes %5d lanes %2d warps %2d : issue %6lld cycles (%5.0f per copy)  issue+land %6lld\n", bytes, lanes, warps, out[0], (double)out[0] / lanes, out[1]);
    }
    return 0;
}
