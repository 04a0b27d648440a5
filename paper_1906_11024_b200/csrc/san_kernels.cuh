// Device code of the shared-attention decode path (sm_100a).
//
// All four steps are HBM-bound streams over head-major cache panels: one (id, head) panel
// is a contiguous run of 64-element rows, so a warp reads it with 16-byte loads, 512 bytes
// per instruction, several instructions in flight.  Arithmetic is float32 on the CUDA
// cores: one query row against a 64-wide key row is 64 multiply-adds per 128 bytes, far
// under the ridge of any tensor-core tile.
//
// Work is cut into warp-sized items (row = (item, head); span = a run of cache positions).
// Rows longer than one span are finished by whichever warp arrives last at a per-row
// ticket (atomicAdd after __threadfence): nothing ever waits on another warp.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/san.h"

namespace san {

constexpr int kDh = 64;          // d_head
constexpr int kWarpsPerCta = 8;  // warps are independent; a CTA is only a scheduling unit
constexpr int kSub = 128;        // cache positions staged on chip per pass of a warp

enum KernelTag { TAG_APPEND = 1, TAG_WEIGHTS = 2, TAG_APPLY = 3, TAG_AAN = 4, TAG_REORDER = 5, TAG_RESET = 7 };

// Device error word: [0]=status, [1]=kernel tag, [2]=item, [3]=offending value, [4]=limit.
__device__ __forceinline__ void record_error(int* err, int tag, int item, int value, int limit) {
    if (atomicCAS(&err[0], 0, (int)SAN_ERR_DEVICE_CHECK) == 0) {
        err[1] = tag; err[2] = item; err[3] = value; err[4] = limit;
    }
}

// ---------------------------------------------------------------- row geometry per dtype
template <typename T> struct RowGeom;
// Cached bf16 rows are stored with their eight 16-byte chunks permuted: logical chunk c of
// the row at position `pos` sits at chunk c ^ (pos & 7).  A tile of such rows copied
// verbatim into shared memory (rows 128 bytes apart, tile starting at a multiple of 8
// positions) can then be read eight rows at a time by ldmatrix without bank conflicts.
// float32 rows (256 bytes) are stored in natural order.
template <> struct RowGeom<__nv_bfloat16> {
    static constexpr int VEC = 8;   // elements per 16-byte load
    static constexpr int LPR = 8;   // lanes per 64-element row
    static __device__ __forceinline__ int chunk(int c, int pos) { return c ^ (pos & 7); }
};
template <> struct RowGeom<float> {
    static constexpr int VEC = 4;
    static constexpr int LPR = 16;
    static __device__ __forceinline__ int chunk(int c, int) { return c; }
};

__device__ __forceinline__ uint4 ld16_stream(const void* p) {
    // cache rows were written by earlier kernels and are read once: non-coherent path,
    // no L1 allocation
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

template <typename T> __device__ __forceinline__ void unpack16(const uint4& v, float* f);
template <> __device__ __forceinline__ void unpack16<__nv_bfloat16>(const uint4& v, float* f) {
    // a bfloat16 is the upper half of a float32
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
    f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
    f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
}
template <> __device__ __forceinline__ void unpack16<float>(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}

template <typename T> __device__ __forceinline__ uint4 pack16(const float* f);
template <> __device__ __forceinline__ uint4 pack16<__nv_bfloat16>(const float* f) {
    uint4 v;   // round to nearest even
    __nv_bfloat162 a = __floats2bfloat162_rn(f[0], f[1]), b = __floats2bfloat162_rn(f[2], f[3]);
    __nv_bfloat162 c = __floats2bfloat162_rn(f[4], f[5]), d = __floats2bfloat162_rn(f[6], f[7]);
    v.x = *reinterpret_cast<uint32_t*>(&a); v.y = *reinterpret_cast<uint32_t*>(&b);
    v.z = *reinterpret_cast<uint32_t*>(&c); v.w = *reinterpret_cast<uint32_t*>(&d);
    return v;
}
template <> __device__ __forceinline__ uint4 pack16<float>(const float* f) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ------------------------------------------------------------------------------ K1 append
struct AppendParams {
    const char* k_new; const char* v_new;    // source rows
    char* K; char* V;                        // cache plane 0 of each kind
    long long k_plane_bytes, v_plane_bytes;  // bytes between planes
    const int* ids; const int* pos; const int* nrows;
    int n_items, rows_per_item, H, cap_len, max_ids, n_layers, row_bytes;
    int* err;
    short v_plane[SAN_MAX_LAYERS];           // destination V plane per layer of the range
    short k_plane[SAN_MAX_LAYERS];           // destination K plane, or -1
    short k_src[SAN_MAX_LAYERS];             // index of the layer's rows inside k_new
};

// One thread moves 16 bytes.  Unit order (fastest first): 16-byte piece, head, row, item,
// layer, {V,K}; so a warp writes whole rows.
static __global__ void __launch_bounds__(256) append_kernel(const AppendParams p) {
    const int pieces = p.row_bytes >> 4;
    const long long per_kind = (long long)p.n_layers * p.n_items * p.rows_per_item * p.H * pieces;
    long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= 2 * per_kind) return;
    const int is_k = u >= per_kind;
    if (is_k) u -= per_kind;
    const int piece = (int)(u % pieces); u /= pieces;
    const int h = (int)(u % p.H); u /= p.H;
    const int r = (int)(u % p.rows_per_item); u /= p.rows_per_item;
    const int item = (int)(u % p.n_items);
    const int lr = (int)(u / p.n_items);
    const int plane = is_k ? p.k_plane[lr] : p.v_plane[lr];
    if (plane < 0) return;
    const int id = p.ids[item];
    const int pos = p.pos ? p.pos[item] : 0;
    const int nr = p.nrows ? p.nrows[item] : 1;
    const bool reporter = (!is_k && lr == 0 && r == 0 && h == 0 && piece == 0);
    if (id < 0 || id >= p.max_ids) { if (reporter) record_error(p.err, TAG_APPEND, item, id, p.max_ids); return; }
    if (nr < 0 || nr > p.rows_per_item) { if (reporter) record_error(p.err, TAG_APPEND, item, nr, p.rows_per_item); return; }
    if (pos < 0 || pos + nr > p.cap_len) { if (reporter) record_error(p.err, TAG_APPEND, item, pos + nr, p.cap_len); return; }
    if (r >= nr) return;
    const int src_layer = is_k ? p.k_src[lr] : lr;
    const char* src = (is_k ? p.k_new : p.v_new) +
        ((((long long)src_layer * p.n_items + item) * p.rows_per_item + r) * p.H + h) * p.row_bytes + piece * 16;
    const int dst_piece = (p.row_bytes == 128) ? (piece ^ ((pos + r) & 7)) : piece;   // bf16 rows are chunk-permuted
    char* dst = (is_k ? p.K + plane * p.k_plane_bytes : p.V + plane * p.v_plane_bytes) +
        ((((long long)id * p.H + h) * p.cap_len) + pos + r) * p.row_bytes + dst_piece * 16;
    *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
}

// ----------------------------------------------------------------------------- K2 weights
struct WeightsParams {
    const void* q;        // [n_items][nq][H][64]
    const void* K;        // key plane of the block: [max_ids][H][cap_len][64]
    const int* ids; const int* lens;
    float* S; long long ld_s;   // [n_items][nq][H][ld_s]
    int n_items, H, nq, cap_len, max_ids, max_len;
    int nq_total, q0;           // query rows per item in q and S; first of the nq rows this launch covers
    int span_len, n_spans_max;  // positions per warp item; spans per row at max_len
    float* part;                // [row][nq][n_spans_max][2] (max, sum) of split rows
    int* tickets;               // [row]
    int* err;
    float scale_log2e;          // log2(e) / sqrt(d_head): logits are kept in the log2 domain
};

// One warp per (item, head, span).  The key tile is read once and scored against the NQ
// query rows that share it (NQ = 1 for self-attention, = beam for encoder memory).
template <typename T, int NQ>
__global__ void __launch_bounds__(kWarpsPerCta * 32) weights_kernel(const WeightsParams p) {
    using G = RowGeom<T>;
    constexpr int VEC = G::VEC, LPR = G::LPR, RPW = 32 / LPR, UNROLL = 4;
    __shared__ float zs_all[kWarpsPerCta][NQ][kSub];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane / LPR, c = lane % LPR;
    const long long w = (long long)blockIdx.x * kWarpsPerCta + warp;
    const long long total = (long long)p.n_items * p.H * p.n_spans_max;
    if (w >= total) return;
    const int span = (int)(w % p.n_spans_max);
    const long long row = w / p.n_spans_max;
    const int h = (int)(row % p.H), item = (int)(row / p.H);
    const int len = p.lens[item], id = p.ids[item];
    if (id < 0 || id >= p.max_ids) { if (lane == 0 && span == 0 && h == 0) record_error(p.err, TAG_WEIGHTS, item, id, p.max_ids); return; }
    if (len < 1 || len > p.max_len) { if (lane == 0 && span == 0 && h == 0) record_error(p.err, TAG_WEIGHTS, item, len, p.max_len); return; }
    const int j0 = span * p.span_len;
    if (j0 >= len) return;
    const int j1 = min(len, j0 + p.span_len);
    const int n_spans = (len + p.span_len - 1) / p.span_len;
    const int nq = p.nq;

    float qf[NQ][VEC];
#pragma unroll
    for (int qi = 0; qi < NQ; ++qi) {
        if (qi < nq) {
            const T* qp = reinterpret_cast<const T*>(p.q) + (((long long)item * p.nq_total + p.q0 + qi) * p.H + h) * kDh + c * VEC;
            uint4 v = *reinterpret_cast<const uint4*>(qp);
            unpack16<T>(v, qf[qi]);
#pragma unroll
            for (int e = 0; e < VEC; ++e) qf[qi][e] *= p.scale_log2e;
        } else {
#pragma unroll
            for (int e = 0; e < VEC; ++e) qf[qi][e] = 0.f;
        }
    }

    const T* Kp = reinterpret_cast<const T*>(p.K) + (((long long)id * p.H + h) * p.cap_len) * kDh;
    float (*zs)[kSub] = zs_all[warp];
    const bool one_pass = (j1 - j0) <= kSub;   // the whole span fits on chip: softmax from shared memory
    float run_max[NQ];
#pragma unroll
    for (int qi = 0; qi < NQ; ++qi) run_max[qi] = -INFINITY;

    for (int s0 = j0; s0 < j1; s0 += kSub) {
        const int n = min(kSub, j1 - s0);
        // scores of positions s0 .. s0+n-1 into shared memory
        for (int jb = 0; jb < n; jb += RPW * UNROLL) {
            uint4 kv[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int j = jb + u * RPW + g;
                kv[u] = (j < n) ? ld16_stream(Kp + (long long)(s0 + j) * kDh + G::chunk(c, s0 + j) * VEC) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int j = jb + u * RPW + g;
                float kf[VEC];
                unpack16<T>(kv[u], kf);
#pragma unroll
                for (int qi = 0; qi < NQ; ++qi) {
                    float d = 0.f;
#pragma unroll
                    for (int e = 0; e < VEC; ++e) d = fmaf(qf[qi][e], kf[e], d);
#pragma unroll
                    for (int o = LPR / 2; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
                    if (c == 0 && j < n) zs[qi][j] = d;
                }
            }
        }
        __syncwarp();
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) {
            if (qi >= nq) break;
            float m = -INFINITY;
            for (int jj = lane; jj < n; jj += 32) m = fmaxf(m, zs[qi][jj]);
            run_max[qi] = fmaxf(run_max[qi], warp_max(m));
            if (!one_pass) {   // park the raw scores in S; they are turned into weights below
                float* Srow = p.S + (((long long)item * p.nq_total + p.q0 + qi) * p.H + h) * p.ld_s + s0;
                for (int jj = lane; jj < n; jj += 32) Srow[jj] = zs[qi][jj];
            }
        }
        __syncwarp();
    }

    // exp and sum over the span, normalise if the span is the whole row
    const int n_span = j1 - j0;
#pragma unroll
    for (int qi = 0; qi < NQ; ++qi) {
        if (qi >= nq) break;
        float* Srow = p.S + (((long long)item * p.nq_total + p.q0 + qi) * p.H + h) * p.ld_s + j0;
        const float m = run_max[qi];
        float s = 0.f;
        if (one_pass) {
            for (int jj = lane; jj < n_span; jj += 32) { float e = exp2f(zs[qi][jj] - m); zs[qi][jj] = e; s += e; }
        } else {
            for (int jj = lane; jj < n_span; jj += 32) { float e = exp2f(__ldcg(Srow + jj) - m); Srow[jj] = e; s += e; }
        }
        s = warp_sum(s);
        if (n_spans == 1) {
            if (one_pass) { for (int jj = lane; jj < n_span; jj += 32) Srow[jj] = zs[qi][jj] / s; }
            else { for (int jj = lane; jj < n_span; jj += 32) Srow[jj] = Srow[jj] / s; }
        } else {
            if (one_pass) { for (int jj = lane; jj < n_span; jj += 32) Srow[jj] = zs[qi][jj]; }
            if (lane == 0) {
                float* pp = p.part + ((row * nq + qi) * p.n_spans_max + span) * 2;
                pp[0] = m; pp[1] = s;
            }
        }
    }
    if (n_spans == 1) return;

    // split row: the last span to arrive rescales the whole row
    __threadfence();
    __syncwarp();
    int t = 0;
    if (lane == 0) t = atomicAdd(p.tickets + row, 1);
    t = __shfl_sync(0xffffffffu, t, 0);
    if (t != n_spans - 1) return;
    __threadfence();
    for (int qi = 0; qi < nq; ++qi) {
        const float* pp = p.part + ((row * nq + qi) * p.n_spans_max) * 2;
        float m = -INFINITY;
        for (int sp = lane; sp < n_spans; sp += 32) m = fmaxf(m, __ldcg(pp + 2 * sp));
        m = warp_max(m);
        float tot = 0.f;
        for (int sp = lane; sp < n_spans; sp += 32) tot += __ldcg(pp + 2 * sp + 1) * exp2f(__ldcg(pp + 2 * sp) - m);
        tot = warp_sum(tot);
        float* Srow = p.S + (((long long)item * p.nq_total + p.q0 + qi) * p.H + h) * p.ld_s;
        for (int sp = 0; sp < n_spans; ++sp) {
            const float f = exp2f(__ldcg(pp + 2 * sp) - m) / tot;
            const int b = sp * p.span_len, e = min(len, b + p.span_len);
            for (int j = b + lane; j < e; j += 32) Srow[j] = __ldcg(Srow + j) * f;
        }
    }
    if (lane == 0) p.tickets[row] = 0;   // ready for the next launch
}

// ------------------------------------------------------------------------------- K3 apply
struct ApplyParams {
    const float* S; long long ld_s;   // [n_items][nq][H][ld_s]
    const void* V;                    // value plane of the first layer in the call
    long long plane_elems;            // elements between consecutive layers' planes
    const int* ids; const int* pos_begin; const int* pos_end;
    void* out;                        // [n_layers][n_items][nq][H][64]
    int n_items, H, nq, cap_len, max_ids, max_len;
    int nq_total, q0;                 // query rows per item in S and out; first of the nq rows this launch covers
    int n_layers, layers_per_warp;
    int span_len, n_spans_max;
    int accumulate;
    float* part;                      // [layer][row][nq][n_spans_max][64]
    int* tickets;                     // [layer][row]
    int* err;
};

// One warp per (item, head, layer group, span): S of the span is staged in shared memory
// once, then the value panels of every layer of the group are streamed against it.
template <typename T, int NQ>
__global__ void __launch_bounds__(kWarpsPerCta * 32) apply_kernel(const ApplyParams p) {
    using G = RowGeom<T>;
    constexpr int VEC = G::VEC, LPR = G::LPR, RPW = 32 / LPR, UNROLL = 4;
    __shared__ float ss_all[kWarpsPerCta][NQ][kSub];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane / LPR, c = lane % LPR;
    const int n_lgroups = (p.n_layers + p.layers_per_warp - 1) / p.layers_per_warp;
    const long long n_rows = (long long)p.n_items * p.H;
    const long long w = (long long)blockIdx.x * kWarpsPerCta + warp;
    if (w >= n_rows * n_lgroups * p.n_spans_max) return;
    const int span = (int)(w % p.n_spans_max);
    const int lg = (int)((w / p.n_spans_max) % n_lgroups);
    const long long row = w / ((long long)p.n_spans_max * n_lgroups);
    const int h = (int)(row % p.H), item = (int)(row / p.H);
    const int id = p.ids[item];
    const int p0 = p.pos_begin ? p.pos_begin[item] : 0, p1 = p.pos_end[item];
    const bool reporter = (lane == 0 && span == 0 && lg == 0 && h == 0);
    if (id < 0 || id >= p.max_ids) { if (reporter) record_error(p.err, TAG_APPLY, item, id, p.max_ids); return; }
    if (p0 < 0 || p1 < p0 || p1 > p.max_len) { if (reporter) record_error(p.err, TAG_APPLY, item, p1, p.max_len); return; }
    const int range = p1 - p0;
    const int n_spans = max(1, (range + p.span_len - 1) / p.span_len);   // an empty range still writes zeros
    if (span >= n_spans) return;
    const int j0 = p0 + span * p.span_len, j1 = min(p1, j0 + p.span_len);
    const int nq = p.nq;
    float (*ss)[kSub] = ss_all[warp];
    const int l_begin = lg * p.layers_per_warp, l_end = min(p.n_layers, l_begin + p.layers_per_warp);

    for (int l = l_begin; l < l_end; ++l) {
        const T* Vp = reinterpret_cast<const T*>(p.V) + (long long)l * p.plane_elems +
                      (((long long)id * p.H + h) * p.cap_len) * kDh;
        float acc[NQ][VEC];
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi)
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[qi][e] = 0.f;

        for (int s0 = j0; s0 < j1; s0 += kSub) {
            const int n = min(kSub, j1 - s0);
            // stage S once per span; spans longer than the staging buffer re-stage per pass
            if (l == l_begin || (j1 - j0) > kSub) {
                __syncwarp();
                for (int qi = 0; qi < nq; ++qi) {
                    const float* Srow = p.S + (((long long)item * p.nq_total + p.q0 + qi) * p.H + h) * p.ld_s + s0;
                    for (int jj = lane; jj < n; jj += 32) ss[qi][jj] = Srow[jj];
                }
                __syncwarp();
            }
            for (int jb = 0; jb < n; jb += RPW * UNROLL) {
                uint4 vv[UNROLL];
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int j = jb + u * RPW + g;
                    vv[u] = (j < n) ? ld16_stream(Vp + (long long)(s0 + j) * kDh + G::chunk(c, s0 + j) * VEC) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int j = jb + u * RPW + g;
                    if (j < n) {
                        float vf[VEC];
                        unpack16<T>(vv[u], vf);
#pragma unroll
                        for (int qi = 0; qi < NQ; ++qi) {
                            const float s = (qi < nq) ? ss[qi][j] : 0.f;
#pragma unroll
                            for (int e = 0; e < VEC; ++e) acc[qi][e] = fmaf(s, vf[e], acc[qi][e]);
                        }
                    }
                }
            }
        }
        // add up the row groups of the warp
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi)
#pragma unroll
            for (int e = 0; e < VEC; ++e)
#pragma unroll
                for (int o = LPR; o < 32; o <<= 1) acc[qi][e] += __shfl_xor_sync(0xffffffffu, acc[qi][e], o);

        if (n_spans == 1) {
            if (g == 0) {
#pragma unroll
                for (int qi = 0; qi < NQ; ++qi) {
                    if (qi >= nq) break;
                    T* op = reinterpret_cast<T*>(p.out) +
                            ((((long long)l * p.n_items + item) * p.nq_total + p.q0 + qi) * p.H + h) * kDh + c * VEC;
                    if (p.accumulate) {
                        float old[VEC];
                        unpack16<T>(*reinterpret_cast<const uint4*>(op), old);
#pragma unroll
                        for (int e = 0; e < VEC; ++e) acc[qi][e] += old[e];
                    }
                    *reinterpret_cast<uint4*>(op) = pack16<T>(acc[qi]);
                }
            }
            continue;
        }

        // split row: park the partial sums, the last span to arrive adds them in span order
        const long long trow = (long long)l * n_rows + row;
        if (g == 0) {
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) {
                if (qi >= nq) break;
                float* pp = p.part + (((trow * nq + qi) * p.n_spans_max) + span) * kDh + c * VEC;
#pragma unroll
                for (int e = 0; e < VEC; ++e) pp[e] = acc[qi][e];
            }
        }
        __threadfence();
        __syncwarp();
        int t = 0;
        if (lane == 0) t = atomicAdd(p.tickets + trow, 1);
        t = __shfl_sync(0xffffffffu, t, 0);
        if (t != n_spans - 1) continue;
        __threadfence();
        for (int qi = 0; qi < nq; ++qi) {
            const float* pp = p.part + ((trow * nq + qi) * p.n_spans_max) * kDh;
            T* op = reinterpret_cast<T*>(p.out) + ((((long long)l * p.n_items + item) * p.nq_total + p.q0 + qi) * p.H + h) * kDh;
            for (int col = lane; col < kDh; col += 32) {
                float a = 0.f;
                for (int sp = 0; sp < n_spans; ++sp) a += __ldcg(pp + (long long)sp * kDh + col);
                if (p.accumulate) a += (float)op[col];
                op[col] = (T)a;
            }
        }
        if (lane == 0) p.tickets[trow] = 0;
    }
}

// --------------------------------------------------------------------------------- K4 AAN
struct AanParams {
    const void* x; void* out; float* sum;   // sum: [layer][max_ids][d]
    const int* ids; const int* t;
    int n_items, d, max_ids, max_t, n_layers, layer_begin;
    int* err;
};

// One thread per 4 adjacent columns: running sum in float32, output = sum / t.
template <typename T>
__global__ void __launch_bounds__(256) aan_kernel(const AanParams p) {
    const int d4 = p.d >> 2;
    long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= (long long)p.n_layers * p.n_items * d4) return;
    const int c4 = (int)(u % d4); u /= d4;
    const int item = (int)(u % p.n_items);
    const int lr = (int)(u / p.n_items);
    const int id = p.ids[item], t = p.t[item];
    if (id < 0 || id >= p.max_ids) { if (c4 == 0 && lr == 0) record_error(p.err, TAG_AAN, item, id, p.max_ids); return; }
    if (t < 1 || t > p.max_t) { if (c4 == 0 && lr == 0) record_error(p.err, TAG_AAN, item, t, p.max_t); return; }
    const long long io = ((long long)lr * p.n_items + item) * p.d + c4 * 4;
    float xv[4];
    if (sizeof(T) == 2) {
        uint2 raw = *reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(p.x) + io);
        xv[0] = __uint_as_float(raw.x << 16); xv[1] = __uint_as_float(raw.x & 0xffff0000u);
        xv[2] = __uint_as_float(raw.y << 16); xv[3] = __uint_as_float(raw.y & 0xffff0000u);
    } else {
        float4 raw = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.x) + io);
        xv[0] = raw.x; xv[1] = raw.y; xv[2] = raw.z; xv[3] = raw.w;
    }
    float4* sp = reinterpret_cast<float4*>(p.sum + (((long long)(p.layer_begin + lr) * p.max_ids + id) * p.d) + c4 * 4);
    float4 s = (t == 1) ? make_float4(0.f, 0.f, 0.f, 0.f) : *sp;
    s.x += xv[0]; s.y += xv[1]; s.z += xv[2]; s.w += xv[3];
    *sp = s;
    const float ft = (float)t;
    const float o0 = s.x / ft, o1 = s.y / ft, o2 = s.z / ft, o3 = s.w / ft;
    if (sizeof(T) == 2) {
        __nv_bfloat162 a = __floats2bfloat162_rn(o0, o1), b = __floats2bfloat162_rn(o2, o3);
        uint2 r; r.x = *reinterpret_cast<uint32_t*>(&a); r.y = *reinterpret_cast<uint32_t*>(&b);
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out) + io) = r;
    } else {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + io) = make_float4(o0, o1, o2, o3);
    }
}

// Zeroes the running sums of the listed sequences in every layer: one thread per 16 bytes.
struct ResetParams {
    float* sum;                    // [layer][max_ids][d]
    const int* ids;
    int n_items, d, max_ids, n_layers;
    int* err;
};

static __global__ void __launch_bounds__(256) aan_reset_kernel(const ResetParams p) {
    const int d4 = p.d >> 2;
    long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= (long long)p.n_layers * p.n_items * d4) return;
    const int c4 = (int)(u % d4); u /= d4;
    const int item = (int)(u % p.n_items);
    const int layer = (int)(u / p.n_items);
    const int id = p.ids[item];
    if (id < 0 || id >= p.max_ids) { if (c4 == 0 && layer == 0) record_error(p.err, TAG_RESET, item, id, p.max_ids); return; }
    reinterpret_cast<float4*>(p.sum + ((long long)layer * p.max_ids + id) * p.d)[c4] = make_float4(0.f, 0.f, 0.f, 0.f);
}

}  // namespace san
