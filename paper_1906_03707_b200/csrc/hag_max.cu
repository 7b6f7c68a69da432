// Element-wise max aggregation (the GraphSAGE-P row of Table 1) over the same HAG:
// max is associative and commutative (a set Aggregate, Section 3.1), so Algorithm 2
// holds with max in place of the sum, and by the cover condition of Theorem 2 every
// in-neighbour reaches its node along exactly one path.  Forward: pair kernel for
// the shallow levels, one gather for the expanded deep levels, one gather over the
// residual rows.  Backward: a component of the gradient of a node goes to the sources
// whose value equals the node's maximum; evaluated as a gather over the transposed
// HAG (no atomics, fixed summation order), two row loads per entry: the
// destination's maximum and its gradient.
//
// One warp per row, LPR lanes per row chunk of 16 bytes, 32/LPR lane groups on
// alternate entries, ids read 32 at a time and handed round by shuffle.  Rows are
// not split here (a row of a thousand entries is walked by one warp).
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <limits>

#include "hag.h"
#include "hag_internal.h"
#include "hag_kernels.cuh"
#include "hag_launch.h"

namespace {

using hagk::Chunk;
using hagk::kThreads;
using hagk::kWarps;
using hagk::Tables;

struct MaxArgs {
    const int32_t *row_ptr;   // indexed by absolute row id
    const int32_t *idx;
    int32_t row_begin, row_count;
    int32_t n_prim;           // ids below: graph nodes (rows of T); from it on: aggregation nodes (fp32 rows)
    int32_t D;
    // forward: values of the sources.  backward: maxima of the destinations (forward output / kept a-hat rows)
    const void *val_prim;
    const float *val_sec;
    // backward only: gradients of the destinations, and this row's own value
    const void *grad_prim;
    const float *grad_sec;
    const void *own_prim;
    const float *own_sec;
    void *out;
    int32_t out_is_f32;
    int32_t out_row_offset;
    const int32_t *order;     // several-rows-per-warp kernels: the row taking the place of absolute row r, or null
};

struct PairMaxArgs {
    const int32_t *agg_in;
    int32_t first, count;
    const void *z;
    float *ahat;
    int32_t n, D;
};

// Launch shapes from a sweep on B200 (loads or entries in flight per lane, resident CTAs per SM):
// more resident warps beat more loads per warp, as for the sum kernels.
//   fp32: forward 4 loads x 10 CTAs, backward 2 entries x 10 CTAs; bf16: forward 4 x 12 (raw word groups: 4 registers
//   per load in flight), backward 4 x 8 (a maximum and a gradient word group per entry).
#define HAG_MAX_SHAPES 4, 10, 2, 10, 4, 12, 4, 8
template <typename T> struct MaxShape;
template <int FL, int FB, int BE, int BB, int HFL, int HFB, int HBE, int HBB> struct MaxShapeTable {
    static constexpr int f32[4] = {FL, FB, BE, BB};
    static constexpr int bf16[4] = {HFL, HFB, HBE, HBB};
};
using MaxShapes = MaxShapeTable<HAG_MAX_SHAPES>;
template <> struct MaxShape<float> {
    // 512-byte rows and wider: 8 loads x 8 CTAs (cfg 3 forward 0.86 -> 0.74 ms against 4 x 10; 16 x 5: 0.86, 8 x 7: 0.77)
    static constexpr __host__ __device__ int fwd_loads(int lpr) { return lpr == 32 ? 8 : MaxShapes::f32[0]; }
    static constexpr int fwd_blocks(int lpr) { return lpr == 32 ? 8 : MaxShapes::f32[1]; }
    static constexpr int kBwdEntries = MaxShapes::f32[2];
    // 512-byte rows and wider: the unchecked loop body needs the registers of one CTA fewer, or it spills
    static constexpr int bwd_blocks(int lpr) { return lpr == 32 ? MaxShapes::f32[3] - 1 : MaxShapes::f32[3]; }
};
template <> struct MaxShape<__nv_bfloat16> {
    static constexpr __host__ __device__ int fwd_loads(int) { return MaxShapes::bf16[0]; }
    static constexpr int fwd_blocks(int) { return MaxShapes::bf16[1]; }
    static constexpr int kBwdEntries = MaxShapes::bf16[2];
    static constexpr int bwd_blocks(int) { return MaxShapes::bf16[3]; }
};

// Packed maximum of two bf16 pairs (one instruction for two values; exact, as every maximum is).
__device__ __forceinline__ uint32_t max_bf16x2(uint32_t x, uint32_t y) {
    const __nv_bfloat162 r = __hmax2(*reinterpret_cast<const __nv_bfloat162 *>(&x), *reinterpret_cast<const __nv_bfloat162 *>(&y));
    return *reinterpret_cast<const uint32_t *>(&r);
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {      // exact for values that are bf16 already
    const __nv_bfloat162 r = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&r);
}

// max over the entries [b, e) of one row by the whole warp (`first`: the row's first 32 ids, one per lane).
template <typename T, int LPR>
__device__ __forceinline__ void max_row(const MaxArgs &a, int32_t row, int32_t b, int32_t e, int32_t first, int lane) {
    constexpr int E = Chunk<T>::kElems;
    constexpr int G = 32 / LPR;
    constexpr int U = MaxShape<T>::fwd_loads(LPR) < LPR ? MaxShape<T>::fwd_loads(LPR) : LPR;
    constexpr unsigned FULL = 0xffffffffu;
    const int slice = lane / LPR, gl = lane % LPR;
    const int n_chunks = a.D / E;
    const float ninf = __int_as_float(0xff800000);      // -infinity: the neutral element of max
    for (int c0 = 0; c0 < n_chunks; c0 += LPR) {
        const int chunk = c0 + gl;
        const bool live = chunk < n_chunks;
        const Tables<T> tab(a.val_prim, a.val_sec, a.n_prim, a.D, live ? chunk : 0);
        int32_t mine = (c0 == 0) ? first : ((b + lane < e) ? __ldg(a.idx + b + lane) : -1);
        if constexpr (E == 8) {
            // bf16 storage: the maximum is taken on the raw bf16 pairs (max.bf16x2: 4 instructions per 16 bytes, no
            // widening), U raw word groups in flight.  The ids of a row ascend, so the bf16 rows (the first n_p entries
            // of a batch) and the fp32 rows of aggregation nodes (whose values are bf16 values) have a loop each.
            constexpr uint32_t kNinf2 = 0xff80ff80u;
            uint32_t m[4] = {kNinf2, kNinf2, kNinf2, kNinf2};
            for (int32_t base = b; base < e; base += 32) {
                const int32_t cur = mine;
                const int32_t nb = base + 32;
                mine = (nb + lane < e) ? __ldg(a.idx + nb + lane) : -1;
                const int cnt = min(32, e - base);
                const int n_p = __popc(__ballot_sync(FULL, cur >= 0 && cur < a.n_prim));
#pragma unroll
                for (int k = 0; k < LPR; k += U) {
                    if (k * G < n_p) {
                        uint4 raw[U];
                        if ((k + U) * G <= n_p) {       // a full group: no checks (lanes beyond the row width read chunk 0, never stored)
#pragma unroll
                            for (int u = 0; u < U; ++u)
                                raw[u] = hagk::ld_u4(tab.prim + size_t(uint32_t(__shfl_sync(FULL, cur, (k + u) * G + slice))) * tab.prim_row_bytes);
                        } else {
#pragma unroll
                            for (int u = 0; u < U; ++u) {
                                const int32_t id = __shfl_sync(FULL, cur, (k + u) * G + slice);
                                raw[u] = ((k + u) * G + slice < n_p && live) ? hagk::ld_u4(tab.prim + size_t(uint32_t(id)) * tab.prim_row_bytes)
                                                                             : make_uint4(kNinf2, kNinf2, kNinf2, kNinf2);
                            }
                        }
#pragma unroll
                        for (int u = 0; u < U; ++u) {
                            m[0] = max_bf16x2(m[0], raw[u].x);
                            m[1] = max_bf16x2(m[1], raw[u].y);
                            m[2] = max_bf16x2(m[2], raw[u].z);
                            m[3] = max_bf16x2(m[3], raw[u].w);
                        }
                    }
                }
                for (int j0 = n_p; j0 < cnt; j0 += G) {
                    const int j = j0 + slice;
                    const int32_t id = __shfl_sync(FULL, cur, j < cnt ? j : 0);
                    if (j < cnt && live) {
                        const char *p = tab.sec + size_t(uint32_t(id)) * tab.sec_row_bytes;
                        const float4 q0 = hagk::ld_f4(p), q1 = hagk::ld_f4(p + 16);
                        m[0] = max_bf16x2(m[0], pack_bf16x2(q0.x, q0.y));
                        m[1] = max_bf16x2(m[1], pack_bf16x2(q0.z, q0.w));
                        m[2] = max_bf16x2(m[2], pack_bf16x2(q1.x, q1.y));
                        m[3] = max_bf16x2(m[3], pack_bf16x2(q1.z, q1.w));
                    }
                }
            }
#pragma unroll
            for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
                for (int i = 0; i < 4; ++i) m[i] = max_bf16x2(m[i], __shfl_xor_sync(FULL, m[i], off));
            if (live && slice == 0) {
                float acc[E];
                hagk::bf16x8_to_f32(make_uint4(m[0], m[1], m[2], m[3]), acc);
                if (e == b) {                 // empty neighbourhood: zero row
#pragma unroll
                    for (int j = 0; j < E; ++j) acc[j] = 0.0f;
                }
                hagk::store_chunk<T>(a.out, a.out_is_f32, a.D, row - a.out_row_offset, chunk, acc);
            }
        } else {
            float acc[E];
#pragma unroll
            for (int j = 0; j < E; ++j) acc[j] = ninf;
            for (int32_t base = b; base < e; base += 32) {
                const int32_t cur = mine;
                const int32_t nb = base + 32;
                mine = (nb + lane < e) ? __ldg(a.idx + nb + lane) : -1;
                const int cnt = min(32, e - base);
#pragma unroll
                for (int k = 0; k < LPR; k += U) {
                    if (k * G < cnt) {
                        float v[U][E];
                        if ((k + U) * G <= cnt) {       // a full group: no checks, no fill (lanes beyond the row width read chunk 0, never stored)
#pragma unroll
                            for (int u = 0; u < U; ++u) tab.load(__shfl_sync(FULL, cur, (k + u) * G + slice), v[u]);
                        } else {
#pragma unroll
                            for (int u = 0; u < U; ++u) {
                                const int32_t id = __shfl_sync(FULL, cur, (k + u) * G + slice);
                                if (id >= 0 && live) {
                                    tab.load(id, v[u]);
                                } else {
#pragma unroll
                                    for (int j = 0; j < E; ++j) v[u][j] = ninf;
                                }
                            }
                        }
#pragma unroll
                        for (int u = 0; u < U; ++u)
#pragma unroll
                            for (int j = 0; j < E; ++j) acc[j] = fmaxf(acc[j], v[u][j]);
                    }
                }
            }
#pragma unroll
            for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
                for (int j = 0; j < E; ++j) acc[j] = fmaxf(acc[j], __shfl_xor_sync(FULL, acc[j], off));
            if (live && slice == 0) {
                if (e == b) {                 // empty neighbourhood: zero row
#pragma unroll
                    for (int j = 0; j < E; ++j) acc[j] = 0.0f;
                }
                hagk::store_chunk<T>(a.out, a.out_is_f32, a.D, row - a.out_row_offset, chunk, acc);
            }
        }
    }
}

template <typename T, int LPR>
__global__ void __launch_bounds__(kThreads, MaxShape<T>::fwd_blocks(LPR)) gather_max_kernel(const MaxArgs a) {
    hagk::pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int r_local = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (r_local >= a.row_count) return;
    int32_t row = a.row_begin + r_local;
    if (a.order) row = __ldg(a.order + row);
    const int32_t b = __ldg(a.row_ptr + row), e = __ldg(a.row_ptr + row + 1);
    const int32_t first = (b + lane < e) ? __ldg(a.idx + b + lane) : -1;
    hagk::pdl_wait();
    max_row<T, LPR>(a, row, b, e, first, lane);
}

// Several rows per warp (feature rows of 256 bytes or less), as for the sums: every group of LPR lanes walks a row of its
// own, taken in the list's by-length order, in lock step with the other groups; no value crosses lanes.  Rows are not
// cut into segments here, so a row of more than kMaxSubLong entries is left out of the lock step and walked by the
// whole warp afterwards.
constexpr int32_t kMaxSubLong = 128;

template <typename T, int LPR>
__global__ void __launch_bounds__(kThreads, sizeof(T) == 4 ? 9 : 8) gather_max_sub_kernel(const MaxArgs a) {
    static_assert(LPR < 32, "one row per warp is gather_max_kernel's job");
    hagk::pdl_launch_dependents();
    constexpr int E = Chunk<T>::kElems;
    constexpr int G = 32 / LPR;
    constexpr int U = sizeof(T) == 4 ? 8 : 2;      // fp32: 8 loads x 9 CTAs from a sweep (-7 % against 4 x 10 on cfg 4); bf16 rows are
                                                   // widened to fp32 in flight, 8 registers each
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int item = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (item * G >= a.row_count) return;
    const int slice = lane / LPR, gl = lane % LPR;
    const int32_t r_local = item * G + slice;
    const bool have = r_local < a.row_count;
    int32_t row = a.row_begin + (have ? r_local : 0);
    if (a.order) row = __ldg(a.order + row);
    int32_t b = 0, e = 0;
    if (have) {
        b = __ldg(a.row_ptr + row);
        e = __ldg(a.row_ptr + row + 1);
    }
    const bool is_long = e - b > kMaxSubLong;
    const int32_t len = is_long ? 0 : e - b;
    int32_t mine = (gl < len) ? __ldg(a.idx + b + gl) : -1;
    const int32_t max_len = __reduce_max_sync(FULL, len);
    hagk::pdl_wait();
    const int n_chunks = a.D / E;
    const bool live = gl < n_chunks;
    const float ninf = __int_as_float(0xff800000);
    const Tables<T> tab(a.val_prim, a.val_sec, a.n_prim, a.D, live ? gl : 0);
    float acc[E];
#pragma unroll
    for (int j = 0; j < E; ++j) acc[j] = ninf;
    for (int32_t off = 0; off < max_len; off += LPR) {
        const int32_t cur = mine;
        const int32_t nb = off + LPR + gl;
        mine = (nb < len) ? __ldg(a.idx + b + nb) : -1;
        const int32_t cnt = len - off, max_cnt = max_len - off;
#pragma unroll
        for (int kk = 0; kk < LPR; kk += U) {
            if (kk < max_cnt) {
                float v[U][E];
                if (__all_sync(FULL, kk + U <= cnt)) {
#pragma unroll
                    for (int u = 0; u < U; ++u) tab.load(__shfl_sync(FULL, cur, kk + u, LPR), v[u]);
                } else {
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int32_t id = __shfl_sync(FULL, cur, kk + u, LPR);
                        if (id >= 0 && live) {
                            tab.load(id, v[u]);
                        } else {
#pragma unroll
                            for (int j = 0; j < E; ++j) v[u][j] = ninf;
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u)
#pragma unroll
                    for (int j = 0; j < E; ++j) acc[j] = fmaxf(acc[j], v[u][j]);
            }
        }
    }
    if (have && live && !is_long) {
        if (e == b) {                 // empty neighbourhood: zero row
#pragma unroll
            for (int j = 0; j < E; ++j) acc[j] = 0.0f;
        }
        hagk::store_chunk<T>(a.out, a.out_is_f32, a.D, row - a.out_row_offset, gl, acc);
    }
    // the long rows among this warp's rows, one after the other, by the whole warp
    unsigned todo = __ballot_sync(FULL, is_long && gl == 0);
    while (todo) {
        const int src = __ffs(todo) - 1;
        todo &= todo - 1;
        const int32_t lrow = __shfl_sync(FULL, row, src), lb = __shfl_sync(FULL, b, src), le = __shfl_sync(FULL, e, src);
        max_row<T, LPR>(a, lrow, lb, le, (lb + lane < le) ? __ldg(a.idx + lb + lane) : -1, lane);
    }
}

// a-hat_w = max(a-hat_in0, a-hat_in1) for one level; one lane group per aggregation node.
template <typename T, int LPR>
__global__ void __launch_bounds__(kThreads) pair_max_kernel(const PairMaxArgs p) {
    hagk::pdl_launch_dependents();
    constexpr int E = Chunk<T>::kElems;
    constexpr int G = 32 / LPR;
    const int lane = threadIdx.x & 31;
    const int slice = lane / LPR, gl = lane % LPR;
    const int32_t j = (blockIdx.x * kWarps + (threadIdx.x >> 5)) * G + slice;
    if (j >= p.count) return;
    const int2 in = __ldg(reinterpret_cast<const int2 *>(p.agg_in) + p.first + j);
    hagk::pdl_wait();
    const int n_chunks = p.D / E;
    for (int chunk = gl; chunk < n_chunks; chunk += LPR) {
        const Tables<T> tab(p.z, p.ahat, p.n, p.D, chunk);
        float u[E], v[E];
        tab.load(in.x, u);
        tab.load(in.y, v);
#pragma unroll
        for (int i = 0; i < E; ++i) u[i] = fmaxf(u[i], v[i]);
        hagk::store_chunk<T>(p.ahat, 1, p.D, p.first + j, chunk, u);
    }
}

// acc[0..8) += the gradient words g where the destination's maximum words v equal this row's value words (bf16 pairs
// compared two at a time: ordered equality, +0 == -0, NaN equal to nothing, as for floats; the kept gradient pairs are
// widened by a shift or a mask and added as packed fp32 pairs).
__device__ __forceinline__ void add_where_equal_bf16x8(float *acc, const uint4 &v, const uint4 &g, const uint4 &own) {
    const uint32_t vw[4] = {v.x, v.y, v.z, v.w}, gw[4] = {g.x, g.y, g.z, g.w}, ow[4] = {own.x, own.y, own.z, own.w};
    uint4 kept;
    uint32_t *kw = &kept.x;
#pragma unroll
    for (int i = 0; i < 4; ++i)
        kw[i] = gw[i] & __heq2_mask(*reinterpret_cast<const __nv_bfloat162 *>(&vw[i]), *reinterpret_cast<const __nv_bfloat162 *>(&ow[i]));
    hagk::add_bf16x8<false>(acc, kept, 1.0f);
}

// grad_s[k] = sum over the destinations t of row s with max_t[k] == value_s[k] of grad_t[k].
template <typename T, int LPR>
__device__ __forceinline__ void maxgrad_row(const MaxArgs &a, int32_t row, int32_t b, int32_t e, int32_t first, int lane) {
    constexpr int E = Chunk<T>::kElems;
    constexpr int G = 32 / LPR;
    constexpr int U = MaxShape<T>::kBwdEntries < LPR ? MaxShape<T>::kBwdEntries : LPR;
    constexpr unsigned FULL = 0xffffffffu;
    const int slice = lane / LPR, gl = lane % LPR;
    const int n_chunks = a.D / E;
    for (int c0 = 0; c0 < n_chunks; c0 += LPR) {
        const int chunk = c0 + gl;
        const bool live = chunk < n_chunks;
        const Tables<T> vals(a.val_prim, a.val_sec, a.n_prim, a.D, live ? chunk : 0);
        const Tables<T> grads(a.grad_prim, a.grad_sec, a.n_prim, a.D, live ? chunk : 0);
        const Tables<T> self(a.own_prim, a.own_sec, a.n_prim, a.D, live ? chunk : 0);
        float acc[E];
#pragma unroll
        for (int j = 0; j < E; ++j) acc[j] = 0.0f;
        int32_t mine = (c0 == 0) ? first : ((b + lane < e) ? __ldg(a.idx + b + lane) : -1);
        if constexpr (E == 8) {
            // bf16 storage.  Maxima are bf16 values wherever they are kept, so the comparison runs on bf16 pairs (this
            // row's value packed once); the rows of graph-node destinations stay raw words from the load to the masked
            // add, U entries (a maximum and a gradient word group each) in flight.  The ids of a row ascend: the
            // graph-node destinations are the first n_p entries of a batch, the aggregation nodes (fp32 maxima and fp32
            // gradients) the rest, a loop each.
            uint4 own;
            if (row < a.n_prim) {
                own = hagk::ld_u4(self.prim + size_t(uint32_t(row)) * self.prim_row_bytes);
            } else {
                const char *p = self.sec + size_t(uint32_t(row)) * self.sec_row_bytes;
                const float4 q0 = hagk::ld_f4(p), q1 = hagk::ld_f4(p + 16);
                own = make_uint4(pack_bf16x2(q0.x, q0.y), pack_bf16x2(q0.z, q0.w), pack_bf16x2(q1.x, q1.y), pack_bf16x2(q1.z, q1.w));
            }
            for (int32_t base = b; base < e; base += 32) {
                const int32_t cur = mine;
                const int32_t nb = base + 32;
                mine = (nb + lane < e) ? __ldg(a.idx + nb + lane) : -1;
                const int cnt = min(32, e - base);
                const int n_p = __popc(__ballot_sync(FULL, cur >= 0 && cur < a.n_prim));
#pragma unroll
                for (int k = 0; k < LPR; k += U) {
                    if (k * G < n_p) {
                        uint4 rv[U], rg[U];
                        if ((k + U) * G <= n_p) {       // a full group: no checks (lanes beyond the row width read chunk 0, never stored)
#pragma unroll
                            for (int u = 0; u < U; ++u) {
                                const size_t off = size_t(uint32_t(__shfl_sync(FULL, cur, (k + u) * G + slice))) * vals.prim_row_bytes;
                                rv[u] = hagk::ld_u4(vals.prim + off);
                                rg[u] = hagk::ld_u4(grads.prim + off);
                            }
                        } else {
#pragma unroll
                            for (int u = 0; u < U; ++u) {
                                const int32_t id = __shfl_sync(FULL, cur, (k + u) * G + slice);
                                if ((k + u) * G + slice < n_p && live) {
                                    const size_t off = size_t(uint32_t(id)) * vals.prim_row_bytes;
                                    rv[u] = hagk::ld_u4(vals.prim + off);
                                    rg[u] = hagk::ld_u4(grads.prim + off);
                                } else {
                                    rv[u] = rg[u] = make_uint4(0u, 0u, 0u, 0u);      // a zero gradient adds nothing
                                }
                            }
                        }
#pragma unroll
                        for (int u = 0; u < U; ++u) add_where_equal_bf16x8(acc, rv[u], rg[u], own);
                    }
                }
                for (int j0 = n_p; j0 < cnt; j0 += G) {
                    const int j = j0 + slice;
                    const int32_t id = __shfl_sync(FULL, cur, j < cnt ? j : 0);
                    if (j < cnt && live) {
                        const size_t off = size_t(uint32_t(id)) * vals.sec_row_bytes;
                        const float4 v0 = hagk::ld_f4(vals.sec + off), v1 = hagk::ld_f4(vals.sec + off + 16);
                        const float4 g0 = hagk::ld_f4(grads.sec + off), g1 = hagk::ld_f4(grads.sec + off + 16);
                        const uint32_t ow[4] = {own.x, own.y, own.z, own.w};
                        const uint32_t vw[4] = {pack_bf16x2(v0.x, v0.y), pack_bf16x2(v0.z, v0.w), pack_bf16x2(v1.x, v1.y), pack_bf16x2(v1.z, v1.w)};
                        const float gf[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint32_t m = __heq2_mask(*reinterpret_cast<const __nv_bfloat162 *>(&vw[i]), *reinterpret_cast<const __nv_bfloat162 *>(&ow[i]));
                            acc[2 * i] += (m & 0xffffu) ? gf[2 * i] : 0.0f;
                            acc[2 * i + 1] += (m >> 16) ? gf[2 * i + 1] : 0.0f;
                        }
                    }
                }
            }
        } else {
            float own[E];
            self.load(row, own);
            for (int32_t base = b; base < e; base += 32) {
                const int32_t cur = mine;
                const int32_t nb = base + 32;
                mine = (nb + lane < e) ? __ldg(a.idx + nb + lane) : -1;
                const int cnt = min(32, e - base);
                float part[E];            // two-level sum: one partial per batch of 32 ids
#pragma unroll
                for (int j = 0; j < E; ++j) part[j] = 0.0f;
#pragma unroll
                for (int k = 0; k < LPR; k += U) {
                    if (k * G < cnt) {
                        float tv[U][E], tg[U][E];
                        if ((k + U) * G <= cnt) {       // a full group: no checks, no fill
#pragma unroll
                            for (int u = 0; u < U; ++u) {
                                const int32_t id = __shfl_sync(FULL, cur, (k + u) * G + slice);
                                vals.load(id, tv[u]);
                                grads.load(id, tg[u]);
                            }
                        } else {
#pragma unroll
                            for (int u = 0; u < U; ++u) {
                                const int32_t id = __shfl_sync(FULL, cur, (k + u) * G + slice);
                                if (id >= 0 && live) {
                                    vals.load(id, tv[u]);
                                    grads.load(id, tg[u]);
                                } else {
#pragma unroll
                                    for (int j = 0; j < E; ++j) { tv[u][j] = own[j]; tg[u][j] = 0.0f; }
                                }
                            }
                        }
#pragma unroll
                        for (int u = 0; u < U; ++u)
#pragma unroll
                            for (int j = 0; j < E; ++j) part[j] += (tv[u][j] == own[j]) ? tg[u][j] : 0.0f;
                    }
                }
#pragma unroll
                for (int j = 0; j < E; ++j) acc[j] += part[j];
            }
        }
#pragma unroll
        for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
            for (int j = 0; j < E; ++j) acc[j] += __shfl_xor_sync(FULL, acc[j], off);
        if (live && slice == 0) hagk::store_chunk<T>(a.out, a.out_is_f32, a.D, row - a.out_row_offset, chunk, acc);
    }
}

template <typename T, int LPR>
__global__ void __launch_bounds__(kThreads, MaxShape<T>::bwd_blocks(LPR)) gather_maxgrad_kernel(const MaxArgs a) {
    hagk::pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int r_local = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (r_local >= a.row_count) return;
    int32_t row = a.row_begin + r_local;
    if (a.order) row = __ldg(a.order + row);
    const int32_t b = __ldg(a.row_ptr + row), e = __ldg(a.row_ptr + row + 1);
    const int32_t first = (b + lane < e) ? __ldg(a.idx + b + lane) : -1;
    hagk::pdl_wait();
    maxgrad_row<T, LPR>(a, row, b, e, first, lane);
}

// The backward form of gather_max_sub_kernel: a row per group of LPR lanes, two entries (a maximum row and a gradient
// row each) in flight per lane; sums per batch of LPR ids, then batches.
template <typename T, int LPR>
__global__ void __launch_bounds__(kThreads, sizeof(T) == 4 ? 8 : 6) gather_maxgrad_sub_kernel(const MaxArgs a) {
    static_assert(LPR < 32, "one row per warp is gather_maxgrad_kernel's job");
    hagk::pdl_launch_dependents();
    constexpr int E = Chunk<T>::kElems;
    constexpr int G = 32 / LPR;
    constexpr int U = sizeof(T) == 4 ? 4 : 2;      // entries (a maximum row and a gradient row each) in flight; fp32: 4 x 8 CTAs
                                                   // from a sweep (-2 to -12 % against 2 x 10)
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int item = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (item * G >= a.row_count) return;
    const int slice = lane / LPR, gl = lane % LPR;
    const int32_t r_local = item * G + slice;
    const bool have = r_local < a.row_count;
    int32_t row = a.row_begin + (have ? r_local : 0);
    if (a.order) row = __ldg(a.order + row);
    int32_t b = 0, e = 0;
    if (have) {
        b = __ldg(a.row_ptr + row);
        e = __ldg(a.row_ptr + row + 1);
    }
    const bool is_long = e - b > kMaxSubLong;
    const int32_t len = is_long ? 0 : e - b;
    int32_t mine = (gl < len) ? __ldg(a.idx + b + gl) : -1;
    const int32_t max_len = __reduce_max_sync(FULL, len);
    hagk::pdl_wait();
    const int n_chunks = a.D / E;
    const bool live = gl < n_chunks;
    const Tables<T> vals(a.val_prim, a.val_sec, a.n_prim, a.D, live ? gl : 0);
    const Tables<T> grads(a.grad_prim, a.grad_sec, a.n_prim, a.D, live ? gl : 0);
    float own[E], acc[E];
    {
        const Tables<T> self(a.own_prim, a.own_sec, a.n_prim, a.D, live ? gl : 0);
        self.load(row, own);
    }
#pragma unroll
    for (int j = 0; j < E; ++j) acc[j] = 0.0f;
    for (int32_t off = 0; off < max_len; off += LPR) {
        const int32_t cur = mine;
        const int32_t nb = off + LPR + gl;
        mine = (nb < len) ? __ldg(a.idx + b + nb) : -1;
        const int32_t cnt = len - off, max_cnt = max_len - off;
        float part[E];
#pragma unroll
        for (int j = 0; j < E; ++j) part[j] = 0.0f;
#pragma unroll
        for (int kk = 0; kk < LPR; kk += U) {
            if (kk < max_cnt) {
                float tv[U][E], tg[U][E];
                if (__all_sync(FULL, kk + U <= cnt)) {
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int32_t id = __shfl_sync(FULL, cur, kk + u, LPR);
                        vals.load(id, tv[u]);
                        grads.load(id, tg[u]);
                    }
                } else {
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int32_t id = __shfl_sync(FULL, cur, kk + u, LPR);
                        if (id >= 0 && live) {
                            vals.load(id, tv[u]);
                            grads.load(id, tg[u]);
                        } else {
#pragma unroll
                            for (int j = 0; j < E; ++j) { tv[u][j] = own[j]; tg[u][j] = 0.0f; }
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u)
#pragma unroll
                    for (int j = 0; j < E; ++j) part[j] += (tv[u][j] == own[j]) ? tg[u][j] : 0.0f;
            }
        }
#pragma unroll
        for (int j = 0; j < E; ++j) acc[j] += part[j];
    }
    if (have && live && !is_long) hagk::store_chunk<T>(a.out, a.out_is_f32, a.D, row - a.out_row_offset, gl, acc);
    unsigned todo = __ballot_sync(FULL, is_long && gl == 0);
    while (todo) {
        const int src = __ffs(todo) - 1;
        todo &= todo - 1;
        const int32_t lrow = __shfl_sync(FULL, row, src), lb = __shfl_sync(FULL, b, src), le = __shfl_sync(FULL, e, src);
        maxgrad_row<T, LPR>(a, lrow, lb, le, (lb + lane < le) ? __ldg(a.idx + lb + lane) : -1, lane);
    }
}

using DeviceScope = hagl::DeviceGuard;
using hagl::aligned16;

template <typename Args>
cudaError_t launch(void (*kernel)(Args), int64_t warps, const Args &args, cudaStream_t s) {
    return hagl::launch_pdl(kernel, unsigned((warps + kWarps - 1) / kWarps), unsigned(kThreads), args, s);
}

inline int lanes_for(int n_chunks) { return hagl::lanes_per_row(n_chunks); }

// Launches large enough to give every resident warp a group of rows take several rows per warp (as the sums do).
constexpr int64_t kSubMinWarps = 4096;

template <typename T, int LPR>
cudaError_t launch_rows_lpr(bool grad, const MaxArgs &a, cudaStream_t s) {
    if constexpr (LPR < 32) {
        constexpr int G = 32 / LPR;
        if (a.row_count >= kSubMinWarps * G) {
            const int64_t items = (int64_t(a.row_count) + G - 1) / G;
            return grad ? launch(gather_maxgrad_sub_kernel<T, LPR>, items, a, s) : launch(gather_max_sub_kernel<T, LPR>, items, a, s);
        }
    }
    return grad ? launch(gather_maxgrad_kernel<T, LPR>, a.row_count, a, s) : launch(gather_max_kernel<T, LPR>, a.row_count, a, s);
}

template <typename T>
cudaError_t launch_rows(bool grad, MaxArgs a, const seg_set &set, bool agg_rows, cudaStream_t s) {
    if (a.row_count <= 0) return cudaSuccess;
    const int lpr = lanes_for(a.D / Chunk<T>::kElems);
    // the row order: for the several-rows-per-warp kernels, and for launches of aggregation-node rows large enough for
    // the order of their neighbourhoods to matter
    const bool sub = lpr < 32 && a.row_count >= kSubMinWarps * (32 / lpr);
    a.order = (set.d_order && (sub || (agg_rows && a.row_count >= kOrderNearRows))) ? set.d_order - set.order_first_row : nullptr;
    switch (lpr) {
        case 4: return launch_rows_lpr<T, 4>(grad, a, s);
        case 8: return launch_rows_lpr<T, 8>(grad, a, s);
        case 16: return launch_rows_lpr<T, 16>(grad, a, s);
        default: return launch_rows_lpr<T, 32>(grad, a, s);
    }
}

template <typename T>
cudaError_t launch_pair_level(const PairMaxArgs &p, cudaStream_t s) {
    if (p.count <= 0) return cudaSuccess;
    const int lpr = lanes_for(p.D / Chunk<T>::kElems);
    const int64_t warps = (int64_t(p.count) + (32 / lpr) - 1) / (32 / lpr);
    switch (lpr) {
        case 4: return launch(pair_max_kernel<T, 4>, warps, p, s);
        case 8: return launch(pair_max_kernel<T, 8>, warps, p, s);
        case 16: return launch(pair_max_kernel<T, 16>, warps, p, s);
        default: return launch(pair_max_kernel<T, 32>, warps, p, s);
    }
}

hag_status check(const hag *h, hag_dtype dtype, int32_t D) {
    if (!h) return HAG_ERR_NULL;
    if (dtype != HAG_F32 && dtype != HAG_BF16) return HAG_ERR_DTYPE;
    if (D <= 0) return HAG_ERR_ARG;
    if ((size_t(D) * (dtype == HAG_F32 ? 4 : 2)) % 16 != 0) return HAG_ERR_ALIGN;
    if (h->device < 0) return HAG_ERR_NOT_ON_DEVICE;
    return HAG_OK;
}

constexpr int32_t kAllPrim = std::numeric_limits<int32_t>::max();

template <typename T>
hag_status max_fwd(hag *h, bool use_hag, int32_t D, const void *z, void *out, float *ahat, cudaStream_t s) {
    const hag_device_arrays &d = h->d;
    int32_t launches = 0;
    MaxArgs a{};
    a.D = D;
    a.val_prim = z;
    a.n_prim = kAllPrim;
    if (use_hag && h->num_agg > 0) {
        for (int32_t l = 1; l <= h->fwd_cut; ++l) {        // Algorithm 2 lines 5-6, level by level
            PairMaxArgs p{d.agg_in, int32_t(h->level_ptr[l - 1]), int32_t(h->level_ptr[l] - h->level_ptr[l - 1]), z, ahat, h->n, D};
            if (p.count <= 0) continue;
            if (launch_pair_level<T>(p, s) != cudaSuccess) return HAG_ERR_CUDA;
            ++launches;
        }
        const int32_t j0 = int32_t(h->level_ptr[h->fwd_cut]);
        if (j0 < h->num_agg) {                             // the deeper nodes from their expansion: max over the cover
            MaxArgs t = a;
            t.row_ptr = d.ftail_ptr - (h->n + j0);
            t.idx = d.ftail_idx;
            t.row_begin = h->n + j0;
            t.row_count = h->num_agg - j0;
            t.val_sec = ahat;
            t.n_prim = h->n;
            t.out = ahat;
            t.out_is_f32 = 1;
            t.out_row_offset = h->n;
            if (launch_rows<T>(false, t, h->seg_ftail, true, s) != cudaSuccess) return HAG_ERR_CUDA;
            ++launches;
        }
        a.val_sec = ahat;
        a.n_prim = h->n;
    }
    a.row_ptr = use_hag ? d.res_ptr : d.csr_ptr;           // lines 7-8
    a.idx = use_hag ? d.res_idx : d.csr_idx;
    a.row_begin = 0;
    a.row_count = h->n;
    a.out = out;
    if (h->n > 0) {
        if (launch_rows<T>(false, a, use_hag ? h->seg_res : h->seg_csr, false, s) != cudaSuccess) return HAG_ERR_CUDA;
        ++launches;
    }
    h->last_launches = launches;
    return HAG_OK;
}

template <typename T>
hag_status max_bwd(hag *h, bool use_hag, int32_t D, const void *z, const void *out, const float *ahat, const void *g,
                   void *gz, float *ghat, cudaStream_t s) {
    const hag_device_arrays &d = h->d;
    int32_t launches = 0;
    MaxArgs a{};
    a.D = D;
    a.val_prim = out;         // a graph-node destination: its forward output and its incoming gradient
    a.grad_prim = g;
    a.own_prim = z;
    a.n_prim = kAllPrim;
    if (use_hag && h->num_agg > 0) {
        a.val_sec = ahat;     // an aggregation-node destination: its kept maximum and its computed gradient
        a.grad_sec = ghat;
        a.own_sec = ahat;
        a.n_prim = h->n;
        const int32_t j0 = int32_t(h->level_ptr[h->bwd_cut]);
        if (j0 < h->num_agg) {                             // deep nodes straight from the graph nodes that use them
            MaxArgs t = a;
            t.row_ptr = d.btail_ptr - (h->n + j0);
            t.idx = d.btail_idx;
            t.row_begin = h->n + j0;
            t.row_count = h->num_agg - j0;
            t.out = ghat;
            t.out_is_f32 = 1;
            t.out_row_offset = h->n;
            if (launch_rows<T>(true, t, h->seg_btail, true, s) != cudaSuccess) return HAG_ERR_CUDA;
            ++launches;
        }
        for (int32_t l = h->bwd_cut; l >= 1; --l) {
            MaxArgs lv = a;
            lv.row_ptr = d.t_ptr;
            lv.idx = d.t_idx;
            lv.row_begin = h->n + int32_t(h->level_ptr[l - 1]);
            lv.row_count = int32_t(h->level_ptr[l] - h->level_ptr[l - 1]);
            lv.out = ghat;
            lv.out_is_f32 = 1;
            lv.out_row_offset = h->n;
            if (lv.row_count <= 0) continue;
            if (launch_rows<T>(true, lv, h->seg_t, true, s) != cudaSuccess) return HAG_ERR_CUDA;
            ++launches;
        }
    }
    a.row_ptr = use_hag ? d.t_ptr : d.csr_t_ptr;
    a.idx = use_hag ? d.t_idx : d.csr_t_idx;
    a.row_begin = 0;
    a.row_count = h->n;
    a.out = gz;
    if (h->n > 0) {
        if (launch_rows<T>(true, a, use_hag ? h->seg_t : h->seg_csr_t, false, s) != cudaSuccess) return HAG_ERR_CUDA;
        ++launches;
    }
    h->last_launches = launches;
    return HAG_OK;
}

hag_status run_fwd(const hag_t *hc, bool use_hag, hag_dtype dtype, int32_t D, const void *z, void *out, void *ws, void *stream) {
    hag_status st = check(hc, dtype, D);
    if (st != HAG_OK) return st;
    if (!z || !out) return HAG_ERR_NULL;
    if (!aligned16(z) || !aligned16(out)) return HAG_ERR_ALIGN;
    if (z == out) return HAG_ERR_ARG;
    hag *h = const_cast<hag *>(hc);
    if (use_hag && h->num_agg > 0) {
        if (!ws) return HAG_ERR_WORKSPACE;
        if (!aligned16(ws)) return HAG_ERR_ALIGN;
    }
    DeviceScope scope(h->device);
    if (!scope.ok) { cudaGetLastError(); return HAG_ERR_CUDA; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = dtype == HAG_F32 ? max_fwd<float>(h, use_hag, D, z, out, static_cast<float *>(ws), s)
                          : max_fwd<__nv_bfloat16>(h, use_hag, D, z, out, static_cast<float *>(ws), s);
    if (st != HAG_OK) cudaGetLastError();
    return st;
}

hag_status run_bwd(const hag_t *hc, bool use_hag, hag_dtype dtype, int32_t D, const void *z, const void *out, const void *fwd_ws,
                   const void *g, void *gz, void *ws, void *stream) {
    hag_status st = check(hc, dtype, D);
    if (st != HAG_OK) return st;
    if (!z || !out || !g || !gz) return HAG_ERR_NULL;
    if (!aligned16(z) || !aligned16(out) || !aligned16(g) || !aligned16(gz)) return HAG_ERR_ALIGN;
    if (gz == z || gz == out || gz == g) return HAG_ERR_ARG;
    hag *h = const_cast<hag *>(hc);
    if (use_hag && h->num_agg > 0) {
        if (!ws || !fwd_ws) return HAG_ERR_WORKSPACE;
        if (!aligned16(ws) || !aligned16(fwd_ws)) return HAG_ERR_ALIGN;
        if (ws == fwd_ws) return HAG_ERR_ARG;
    }
    DeviceScope scope(h->device);
    if (!scope.ok) { cudaGetLastError(); return HAG_ERR_CUDA; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = dtype == HAG_F32
             ? max_bwd<float>(h, use_hag, D, z, out, static_cast<const float *>(fwd_ws), g, gz, static_cast<float *>(ws), s)
             : max_bwd<__nv_bfloat16>(h, use_hag, D, z, out, static_cast<const float *>(fwd_ws), g, gz, static_cast<float *>(ws), s);
    if (st != HAG_OK) cudaGetLastError();
    return st;
}

}  // namespace

extern "C" size_t hag_max_workspace_bytes(const hag_t *h, int32_t D) {
    if (!h || D <= 0) return 0;
    return size_t(h->num_agg) * size_t(D) * sizeof(float);
}

extern "C" hag_status hag_max_fwd(const hag_t *h, hag_dtype dtype, int32_t D, const void *z, void *out, void *workspace,
                                  void *cuda_stream) {
    return run_fwd(h, true, dtype, D, z, out, workspace, cuda_stream);
}

extern "C" hag_status hag_max_bwd(const hag_t *h, hag_dtype dtype, int32_t D, const void *z, const void *out,
                                  const void *fwd_workspace, const void *grad_out, void *grad_z, void *workspace,
                                  void *cuda_stream) {
    return run_bwd(h, true, dtype, D, z, out, fwd_workspace, grad_out, grad_z, workspace, cuda_stream);
}

extern "C" hag_status csr_max_fwd(const hag_t *h, hag_dtype dtype, int32_t D, const void *z, void *out, void *cuda_stream) {
    return run_fwd(h, false, dtype, D, z, out, nullptr, cuda_stream);
}

extern "C" hag_status csr_max_bwd(const hag_t *h, hag_dtype dtype, int32_t D, const void *z, const void *out,
                                  const void *grad_out, void *grad_z, void *cuda_stream) {
    return run_bwd(h, false, dtype, D, z, out, nullptr, grad_out, grad_z, nullptr, cuda_stream);
}
