// Device kernels of the HAG aggregation path (sm_100a).
//
// Everything here is a row gather-sum bounded by memory traffic, so the design
// is about wide coalesced loads and enough of them in flight:
//   * a group of LPR lanes (4..32, a power of two) owns one output row; lane i
//     owns the 16-byte chunk i of the row (4 fp32 or 8 bf16 features), so one
//     load instruction of the group reads one contiguous feature row;
//   * neighbour ids are read coalesced, LPR at a time, and handed round with
//     shuffles; UNROLL row loads are issued back to back before any add, and
//     the next batch of ids is fetched before the current one is consumed;
//   * sums are fp32 in NACC independent accumulators combined at the end in a
//     fixed order: no atomics, same bits every run;
//   * a source id below n_prim reads the primary table (the layer input, fp32
//     or bf16); an id at or above it reads the fp32 rows of the aggregation
//     nodes.  One kernel therefore serves Algorithm 2's final loop, the plain
//     GNN-graph, and every step of the backward pass over the transposed HAG.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace hagk {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct GatherArgs {
    const int32_t *row_ptr;   // CSR pointers, indexed by absolute row id
    const int32_t *idx;       // source ids
    int32_t row_begin;        // first absolute row id handled by this launch
    int32_t row_count;
    const void *prim;         // primary source table, n_prim x D of T
    const float *sec;         // secondary source table, fp32, row (id - n_prim)
    int32_t n_prim;
    const float *src_scale;   // optional per-source factor for primary rows (backward of mean)
    const float *dst_scale;   // optional per-destination factor, indexed by absolute row id
    void *out;                // T rows (out_is_f32 == 0) or fp32 rows (out_is_f32 == 1)
    int32_t out_row_offset;   // absolute row r is written to output row r - out_row_offset
    int32_t out_is_f32;
    int32_t D;
};

template <typename T> struct Chunk;
template <> struct Chunk<float> { static constexpr int kElems = 4; };
template <> struct Chunk<__nv_bfloat16> { static constexpr int kElems = 8; };

__device__ __forceinline__ float4 ld_f4(const void *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }
__device__ __forceinline__ uint4 ld_u4(const void *p) { return __ldg(reinterpret_cast<const uint4 *>(p)); }

__device__ __forceinline__ void bf16x8_to_f32(const uint4 &v, float *f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

__device__ __forceinline__ uint4 f32x8_to_bf16(const float *f) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t *>(&p);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// One source row chunk -> kElems floats.
template <typename T>
__device__ __forceinline__ void load_chunk(const GatherArgs &a, int32_t id, int chunk, float *v) {
    constexpr int E = Chunk<T>::kElems;
    if constexpr (E == 4) {
        const float *p = (id < a.n_prim) ? reinterpret_cast<const float *>(a.prim) + size_t(id) * a.D
                                         : a.sec + size_t(id - a.n_prim) * a.D;
        const float4 q = ld_f4(p + chunk * 4);
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
    } else {
        if (id < a.n_prim) {
            const __nv_bfloat16 *p = reinterpret_cast<const __nv_bfloat16 *>(a.prim) + size_t(id) * a.D;
            bf16x8_to_f32(ld_u4(p + chunk * 8), v);
        } else {
            const float *p = a.sec + size_t(id - a.n_prim) * a.D + chunk * 8;
            const float4 q0 = ld_f4(p), q1 = ld_f4(p + 4);
            v[0] = q0.x; v[1] = q0.y; v[2] = q0.z; v[3] = q0.w;
            v[4] = q1.x; v[5] = q1.y; v[6] = q1.z; v[7] = q1.w;
        }
    }
}

template <typename T>
__device__ __forceinline__ void store_chunk(const GatherArgs &a, int32_t out_row, int chunk, const float *v) {
    constexpr int E = Chunk<T>::kElems;
    if (a.out_is_f32) {
        float *p = reinterpret_cast<float *>(a.out) + size_t(out_row) * a.D + chunk * E;
#pragma unroll
        for (int i = 0; i < E; i += 4) *reinterpret_cast<float4 *>(p + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
    } else if constexpr (E == 4) {
        float *p = reinterpret_cast<float *>(a.out) + size_t(out_row) * a.D + chunk * 4;
        __stcs(reinterpret_cast<float4 *>(p), make_float4(v[0], v[1], v[2], v[3]));
    } else {
        __nv_bfloat16 *p = reinterpret_cast<__nv_bfloat16 *>(a.out) + size_t(out_row) * a.D + chunk * 8;
        __stcs(reinterpret_cast<uint4 *>(p), f32x8_to_bf16(v));
    }
}

// out[row] = (dst_scale[row]) * sum_{e in row} (src_scale[id_e]) * table[id_e]
template <typename T, int LPR>
__global__ void __launch_bounds__(kThreads) gather_sum_kernel(const GatherArgs a) {
    constexpr int E = Chunk<T>::kElems;
    constexpr int UNROLL = (LPR >= 8) ? 8 : LPR;
    constexpr int NACC = (E == 4) ? 8 : 4;      // independent partial sums (keeps fp32 error ~ n/NACC ulps)
    constexpr int NA = (NACC < UNROLL) ? NACC : UNROLL;
    constexpr int GROUPS = 32 / LPR;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int sub = lane / LPR;
    const int gl = lane % LPR;
    const unsigned mask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << (sub * LPR));
    const int r_local = (blockIdx.x * kWarps + warp) * GROUPS + sub;
    if (r_local >= a.row_count) return;
    const int32_t row = a.row_begin + r_local;
    const int32_t b = __ldg(a.row_ptr + row), e = __ldg(a.row_ptr + row + 1);
    const int n_chunks = a.D / E;
    const float dscale = a.dst_scale ? __ldg(a.dst_scale + row) : 1.0f;

    for (int c0 = 0; c0 < n_chunks; c0 += LPR) {
        const int chunk = c0 + gl;
        const bool live = chunk < n_chunks;
        float acc[NA][E];
#pragma unroll
        for (int i = 0; i < NA; ++i)
#pragma unroll
            for (int j = 0; j < E; ++j) acc[i][j] = 0.0f;

        int32_t mine = (b + gl < e) ? __ldg(a.idx + b + gl) : -1;
        for (int32_t base = b; base < e; base += LPR) {
            const int32_t cur = mine;
            const int32_t nb = base + LPR;
            mine = (nb + gl < e) ? __ldg(a.idx + nb + gl) : -1;     // next batch of ids, in flight early
            const int cnt = min(LPR, e - base);
#pragma unroll
            for (int k = 0; k < LPR; k += UNROLL) {
                if (k < cnt) {
                    float v[UNROLL][E];
                    float s[UNROLL];
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) {
                        const int32_t id = __shfl_sync(mask, cur, k + u, LPR);
                        s[u] = 1.0f;
                        if (id >= 0 && live) {
                            load_chunk<T>(a, id, chunk, v[u]);
                            if (a.src_scale && id < a.n_prim) s[u] = __ldg(a.src_scale + id);
                        } else {
#pragma unroll
                            for (int j = 0; j < E; ++j) v[u][j] = 0.0f;
                        }
                    }
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u)
#pragma unroll
                        for (int j = 0; j < E; ++j) acc[u % NA][j] = fmaf(v[u][j], s[u], acc[u % NA][j]);
                }
            }
        }
        if (live) {
            float r[E];
#pragma unroll
            for (int j = 0; j < E; ++j) {
                // fixed pairwise combine of the partial sums
                float t[NA];
#pragma unroll
                for (int i = 0; i < NA; ++i) t[i] = acc[i][j];
#pragma unroll
                for (int w = NA / 2; w >= 1; w /= 2)
#pragma unroll
                    for (int i = 0; i < w; ++i) t[i] += t[i + w];
                r[j] = t[0] * dscale;
            }
            store_chunk<T>(a, row - a.out_row_offset, chunk, r);
        }
    }
}

// Level kernel of Algorithm 2 (lines 5-6): every aggregation node of one level is
// the sum of its two inputs.  Nodes [first, first+count) of the level-sorted order;
// inputs with id < n read x (T), others the fp32 rows of earlier levels.
struct PairArgs {
    const int32_t *agg_in;  // [2*num_agg]
    int32_t first, count;
    const void *x;
    float *ahat;            // fp32 rows of the aggregation nodes
    int32_t n;
    int32_t D;
};

template <typename T, int LPR>
__global__ void __launch_bounds__(kThreads) pair_sum_kernel(const PairArgs p) {
    constexpr int E = Chunk<T>::kElems;
    constexpr int GROUPS = 32 / LPR;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int sub = lane / LPR;
    const int gl = lane % LPR;
    const int j_local = (blockIdx.x * kWarps + warp) * GROUPS + sub;
    if (j_local >= p.count) return;
    const int32_t j = p.first + j_local;
    const int2 in = __ldg(reinterpret_cast<const int2 *>(p.agg_in) + j);
    GatherArgs a{};
    a.prim = p.x;
    a.sec = p.ahat;
    a.n_prim = p.n;
    a.D = p.D;
    const int n_chunks = p.D / E;
    for (int chunk = gl; chunk < n_chunks; chunk += LPR) {
        float u[E], v[E];
        load_chunk<T>(a, in.x, chunk, u);
        load_chunk<T>(a, in.y, chunk, v);
        float *o = p.ahat + size_t(j) * p.D + chunk * E;
#pragma unroll
        for (int i = 0; i < E; i += 4)
            *reinterpret_cast<float4 *>(o + i) = make_float4(u[i] + v[i], u[i + 1] + v[i + 1], u[i + 2] + v[i + 2], u[i + 3] + v[i + 3]);
    }
}

}  // namespace hagk
