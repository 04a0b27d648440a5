// Microbenchmark: cycles per operation of dependent chains on one warp (mma.sync m16n8k16 bf16,
// four independent mma chains, shuffle + add, ldmatrix, ld.shared, exp2, fma), with 1, 4 and 16
// warps of a CTA running the same chains.  Used to see what a warp's serial chain of a work item
// costs.  (The ldmatrix rows here are 128 bytes apart without the chunk permutation the caches
// use, so its figure includes an 8-way bank conflict.)
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -o instruction_latency instruction_latency.cu && ./instruction_latency
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__global__ void k(long long* out, float* sink, int warps_active) {
    __shared__ __align__(128) unsigned char sm[8192];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < 2048; i += blockDim.x) ((uint32_t*)sm)[i] = 0x3f803f80u;
    __syncthreads();
    if (warp >= warps_active) return;
    const int N = 64;
    float acc[4] = {0, 0, 0, 0}, acc2[4] = {0,0,0,0}, acc3[4] = {0,0,0,0}, acc4[4] = {0,0,0,0};
    uint32_t a = 0x3f803f80u + lane;
    long long t0 = clock64();
#pragma unroll
    for (int i = 0; i < N; ++i) mma_bf16(acc, a, a, a, a, a, a);
    long long t1 = clock64();
#pragma unroll
    for (int i = 0; i < N / 4; ++i) { mma_bf16(acc, a, a, a, a, a, a); mma_bf16(acc2, a, a, a, a, a, a); mma_bf16(acc3, a, a, a, a, a, a); mma_bf16(acc4, a, a, a, a, a, a); }
    long long t2 = clock64();
    // shuffle chain
    float v = acc[0];
#pragma unroll
    for (int i = 0; i < N; ++i) v += __shfl_xor_sync(0xffffffffu, v, 1 + (i & 15));
    long long t3 = clock64();
    // ldmatrix -> address dependent chain
    uint32_t addr = (uint32_t)__cvta_generic_to_shared(sm) + (lane & 7) * 128;
    uint32_t r0, r1, r2, r3;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
        addr += (r0 & 16);   // r0 = 0x3f803f80 -> & 16 = 0
    }
    long long t4 = clock64();
    // lds chain
    uint32_t ad2 = (uint32_t)__cvta_generic_to_shared(sm) + lane * 4, x;
#pragma unroll
    for (int i = 0; i < N; ++i) { asm volatile("ld.shared.u32 %0, [%1];" : "=r"(x) : "r"(ad2)); ad2 += (x & 16); }
    long long t5 = clock64();
    float e = v;
#pragma unroll
    for (int i = 0; i < N; ++i) e = exp2f(e) * 1e-30f;
    long long t6 = clock64();
    float f = e + 1.f;
#pragma unroll
    for (int i = 0; i < N; ++i) f = fmaf(f, 1.0001f, 0.5f);
    long long t7 = clock64();
    if (lane == 0 && warp == 0 && blockIdx.x == 0) {
        out[0] = (t1 - t0) / N; out[1] = (t2 - t1) / N; out[2] = (t3 - t2) / N; out[3] = (t4 - t3) / N; out[4] = (t5 - t4) / N; out[5] = (t6 - t5) / N; out[6] = (t7 - t6) / N;
    }
    sink[threadIdx.x] = acc[0] + acc2[1] + acc3[2] + acc4[3] + v + r1 + r2 + r3 + x + e + f;
}
int main() {
    long long* out; cudaMallocManaged(&out, 64);
    float* sink; cudaMalloc(&sink, 4096);
    for (int w : {1, 4, 16}) {
        k<<<148, 512>>>(out, sink, w);
        if (cudaDeviceSynchronize() != cudaSuccess) { printf("error\n"); return 1; }
        printf("warps %2d: mma dependent %lld, mma 4 independent chains %lld per mma, shfl+add %lld, ldmatrix dep %lld, lds dep %lld, exp2+mul %lld, fma %lld\n",
               w, out[0], out[1], out[2], out[3], out[4], out[5], out[6]);
    }
    return 0;
}
