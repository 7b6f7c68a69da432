// Graph read-out (the mean-pooling layer of Section 5.1): segmented sums over
// consecutive rows, and the broadcast that is their gradient.  Streaming kernels:
// every row of x is read once (forward) or written once (backward), so the bound
// is HBM bandwidth; one warp owns one graph, LPR lanes cover one row with 16-byte
// loads and the 32/LPR lane groups take alternate rows.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>

#include "hag.h"
#include "hag_kernels.cuh"
#include "hag_launch.h"

namespace {

struct PoolArgs {
    const int32_t *seg_ptr;
    int32_t n_graphs;
    int32_t n_rows;       // backward only
    int32_t D;
    int32_t mean;
    const void *in;
    void *out;
};

constexpr int kPoolLoads = 4;     // row loads in flight per lane
constexpr int kPoolInner = 8;     // groups of loads per partial sum

template <typename T>
__device__ __forceinline__ void load_chunk(const char *p, float *v) {
    if constexpr (hagk::Chunk<T>::kElems == 4) {
        const float4 q = __ldcs(reinterpret_cast<const float4 *>(p));     // read once: streaming
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
    } else {
        hagk::bf16x8_to_f32(__ldcs(reinterpret_cast<const uint4 *>(p)), v);
    }
}

// out_i = s_i * sum of rows seg_ptr[i] .. seg_ptr[i+1]-1.
template <typename T, int LPR>
__global__ void __launch_bounds__(hagk::kThreads) graph_pool_fwd_kernel(const PoolArgs p) {
    hagk::pdl_launch_dependents();
    constexpr int E = hagk::Chunk<T>::kElems;
    constexpr int G = 32 / LPR;
    constexpr int U = kPoolLoads;
    const int lane = threadIdx.x & 31;
    const int seg = blockIdx.x * hagk::kWarps + (threadIdx.x >> 5);
    if (seg >= p.n_graphs) return;
    hagk::pdl_wait();      // seg_ptr is the caller's array: the kernel before this one may have written it
    const int32_t b = p.seg_ptr[seg], e = p.seg_ptr[seg + 1];
    const int slice = lane / LPR, gl = lane % LPR;
    const int n_chunks = p.D / E;
    const size_t row_bytes = size_t(p.D) * sizeof(T);
    const float scale = (p.mean && e > b) ? 1.0f / float(e - b) : 1.0f;
    for (int c0 = 0; c0 < n_chunks; c0 += LPR) {
        const int chunk = c0 + gl;
        const bool live = chunk < n_chunks;
        const char *base = static_cast<const char *>(p.in) + size_t(live ? chunk : 0) * 16;
        float acc[E];
#pragma unroll
        for (int j = 0; j < E; ++j) acc[j] = 0.0f;
        for (int32_t r0 = b; r0 < e; r0 += G * U * kPoolInner) {
            float part[E];
#pragma unroll
            for (int j = 0; j < E; ++j) part[j] = 0.0f;
#pragma unroll 2
            for (int it = 0; it < kPoolInner; ++it) {
                const int32_t r = r0 + it * (G * U) + slice;
                if (r0 + it * (G * U) >= e) break;
                float v[U][E];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int32_t rr = r + u * G;
                    if (rr < e && live) {
                        load_chunk<T>(base + size_t(rr) * row_bytes, v[u]);
                    } else {
#pragma unroll
                        for (int j = 0; j < E; ++j) v[u][j] = 0.0f;
                    }
                }
#pragma unroll
                for (int w = U / 2; w >= 1; w /= 2)
#pragma unroll
                    for (int u = 0; u < w; ++u)
#pragma unroll
                        for (int j = 0; j < E; ++j) v[u][j] += v[u + w][j];
#pragma unroll
                for (int j = 0; j < E; ++j) part[j] += v[0][j];
            }
#pragma unroll
            for (int j = 0; j < E; ++j) acc[j] += part[j];
        }
#pragma unroll
        for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
            for (int j = 0; j < E; ++j) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], off);
        if (live && slice == 0) {
#pragma unroll
            for (int j = 0; j < E; ++j) acc[j] *= scale;
            hagk::store_chunk<T>(p.out, 0, p.D, seg, chunk, acc);
        }
    }
}

// grad_x_v = s_i * grad_out_i for the rows of graph i; the warps of the first and the
// last graph also clear the rows that belong to no graph.
template <typename T, int LPR>
__global__ void __launch_bounds__(hagk::kThreads) graph_pool_bwd_kernel(const PoolArgs p) {
    hagk::pdl_launch_dependents();
    constexpr int E = hagk::Chunk<T>::kElems;
    constexpr int G = 32 / LPR;
    const int lane = threadIdx.x & 31;
    const int seg = blockIdx.x * hagk::kWarps + (threadIdx.x >> 5);
    if (seg > p.n_graphs) return;                       // item n_graphs: the rows after the last graph
    const int slice = lane / LPR, gl = lane % LPR;
    const int n_chunks = p.D / E;
    int32_t b, e, zb = 0, ze = 0;                       // [b, e): rows that get the gradient; [zb, ze): rows cleared
    hagk::pdl_wait();      // seg_ptr is the caller's array: the kernel before this one may have written it
    if (seg < p.n_graphs) {
        b = p.seg_ptr[seg];
        e = p.seg_ptr[seg + 1];
        if (seg == 0) ze = b;
    } else {
        b = e = 0;
        zb = (p.n_graphs > 0) ? p.seg_ptr[p.n_graphs] : 0;
        ze = p.n_rows;
    }
    const float scale = (p.mean && e > b) ? 1.0f / float(e - b) : 1.0f;
    for (int c0 = 0; c0 < n_chunks; c0 += LPR) {
        const int chunk = c0 + gl;
        if (chunk >= n_chunks) continue;
        float v[E];
#pragma unroll
        for (int j = 0; j < E; ++j) v[j] = 0.0f;
        for (int32_t r = zb + slice; r < ze; r += G) hagk::store_chunk<T>(p.out, 0, p.D, r, chunk, v);
        if (e > b) {
            load_chunk<T>(static_cast<const char *>(p.in) + (size_t(seg) * p.D * sizeof(T)) + size_t(chunk) * 16, v);
#pragma unroll
            for (int j = 0; j < E; ++j) v[j] *= scale;
            for (int32_t r = b + slice; r < e; r += G) hagk::store_chunk<T>(p.out, 0, p.D, r, chunk, v);
        }
    }
}

inline int pool_lanes_per_row(int n_chunks) { return hagl::lanes_per_row(n_chunks); }

template <typename Args>
cudaError_t launch_pool(void (*kernel)(Args), int64_t items, const PoolArgs &p, cudaStream_t s) {
    return hagl::launch_pdl(kernel, unsigned((items + hagk::kWarps - 1) / hagk::kWarps), unsigned(hagk::kThreads), p, s);
}

template <typename T, bool BWD>
cudaError_t launch_pool_lpr(int64_t items, const PoolArgs &p, cudaStream_t s) {
    const int n_chunks = p.D / hagk::Chunk<T>::kElems;
    switch (pool_lanes_per_row(n_chunks)) {
        case 4: return BWD ? launch_pool(graph_pool_bwd_kernel<T, 4>, items, p, s) : launch_pool(graph_pool_fwd_kernel<T, 4>, items, p, s);
        case 8: return BWD ? launch_pool(graph_pool_bwd_kernel<T, 8>, items, p, s) : launch_pool(graph_pool_fwd_kernel<T, 8>, items, p, s);
        case 16: return BWD ? launch_pool(graph_pool_bwd_kernel<T, 16>, items, p, s) : launch_pool(graph_pool_fwd_kernel<T, 16>, items, p, s);
        default: return BWD ? launch_pool(graph_pool_bwd_kernel<T, 32>, items, p, s) : launch_pool(graph_pool_fwd_kernel<T, 32>, items, p, s);
    }
}

hag_status pool_check(bool is_bwd, const int32_t *seg_ptr, int32_t n_graphs, int32_t n_rows, hag_reduce reduce, hag_dtype dtype,
                      int32_t D, const void *in, const void *out) {
    if (dtype != HAG_F32 && dtype != HAG_BF16) return HAG_ERR_DTYPE;
    if (D <= 0 || n_graphs < 0 || n_rows < 0) return HAG_ERR_ARG;
    if (reduce != HAG_SUM && reduce != HAG_MEAN) return HAG_ERR_ARG;
    // a matrix without rows may be NULL: the n_graphs x D one when there is no graph, grad_x when n_rows = 0
    if (!seg_ptr || (!in && (n_graphs > 0)) || (!out && (is_bwd ? n_rows > 0 : n_graphs > 0))) return HAG_ERR_NULL;
    const size_t elem = dtype == HAG_F32 ? 4 : 2;
    if ((size_t(D) * elem) % 16 != 0 || (reinterpret_cast<uintptr_t>(in) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u))
        return HAG_ERR_ALIGN;
    if (in && in == out) return HAG_ERR_ARG;
    return HAG_OK;
}

}  // namespace

extern "C" hag_status hag_graph_pool_fwd(const int32_t *seg_ptr, int32_t n_graphs, hag_reduce reduce, hag_dtype dtype,
                                         int32_t D, const void *x, void *out, void *cuda_stream) {
    hag_status st = pool_check(false, seg_ptr, n_graphs, 0, reduce, dtype, D, x, out);
    if (st != HAG_OK) return st;
    if (n_graphs == 0) return HAG_OK;
    PoolArgs p{seg_ptr, n_graphs, 0, D, reduce == HAG_MEAN ? 1 : 0, x, out};
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const cudaError_t err = dtype == HAG_F32 ? launch_pool_lpr<float, false>(n_graphs, p, s)
                                             : launch_pool_lpr<__nv_bfloat16, false>(n_graphs, p, s);
    if (err != cudaSuccess) { cudaGetLastError(); return HAG_ERR_CUDA; }
    return HAG_OK;
}

extern "C" hag_status hag_graph_pool_bwd(const int32_t *seg_ptr, int32_t n_graphs, int32_t n_rows, hag_reduce reduce,
                                         hag_dtype dtype, int32_t D, const void *grad_out, void *grad_x, void *cuda_stream) {
    hag_status st = pool_check(true, seg_ptr, n_graphs, n_rows, reduce, dtype, D, grad_out, grad_x);
    if (st != HAG_OK) return st;
    if (n_rows == 0) return HAG_OK;
    PoolArgs p{seg_ptr, n_graphs, n_rows, D, reduce == HAG_MEAN ? 1 : 0, grad_out, grad_x};
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const int64_t items = int64_t(n_graphs) + 1;        // one extra warp clears the rows after the last graph
    const cudaError_t err = dtype == HAG_F32 ? launch_pool_lpr<float, true>(items, p, s)
                                             : launch_pool_lpr<__nv_bfloat16, true>(items, p, s);
    if (err != cudaSuccess) { cudaGetLastError(); return HAG_ERR_CUDA; }
    return HAG_OK;
}
