// Device kernels of the HAG aggregation path (sm_100a).
//
// Everything here is a row gather-sum bounded by memory traffic, so the design
// is about wide coalesced loads and enough of them in flight:
//   * one warp owns one output row.  A row of D features is n_chunks 16-byte
//     chunks (4 fp32 or 8 bf16 features); LPR = the power of two >= n_chunks
//     (capped at 32) lanes cover one source row with ONE load instruction, and
//     the 32/LPR lane groups ("slices") of the warp take alternate neighbours,
//     so narrow rows still keep all 32 lanes loading distinct data;
//   * neighbour ids are read coalesced, 32 at a time, and handed round with
//     shuffles; the next batch of ids is fetched before the current one is used;
//   * UNROLL row loads per lane are issued back to back, then summed as a
//     balanced tree into a per-batch partial that is folded into the row's
//     accumulator once per 32 ids: the rounding error grows like
//     n/32 + 32/UNROLL + log2(UNROLL) ulps with two accumulators' worth of
//     registers (more resident warps than UNROLL independent partial sums);
//   * slices are combined with butterfly shuffles in a fixed order; no atomics,
//     one writer per output row: same bits every run;
//   * a source id below n_prim reads the primary table (the layer input, fp32
//     or bf16); an id at or above it reads the fp32 rows of the aggregation
//     nodes.  One kernel therefore serves Algorithm 2's final loop, the plain
//     GNN-graph, and every step of the backward pass over the transposed HAG;
//   * bf16 storage: the ids of a row ascend, so its bf16 rows (the layer input)
//     come before its fp32 rows (aggregation nodes).  Each batch of 32 ids is
//     split at that point; the bf16 rows are fetched as raw 16-byte words, kept
//     raw while in flight (4 registers per load, not 8) and widened two at a
//     time straight into packed fp32x2 adds;
//   * every kernel is launched with programmatic stream serialisation: it lets
//     its successor start launching at once and waits for its predecessor's
//     memory only after it has fetched its own (static) row pointers and ids;
//   * besides the launch-per-level kernels there is a single-launch form of a
//     whole pass (fused_pass_kernel, further down), with bounded waits between
//     the phases of the pass.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace hagk {

constexpr int kThreads = 128;
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
    unsigned int *sched;      // persistent kernel only: [0] next row to hand out, [1] finished warps (both zero at launch)
    void *out;                // T rows or fp32 rows; out_is_f32: bit 0 = fp32 rows; bit 1 (host side: selects the SELF
                              // instantiations) = add the row's own primary-table row (times its src_scale)
                              // before scaling: GCN's (a_v + h_v) term
    int32_t out_row_offset;   // absolute row r is written to output row r - out_row_offset
    int32_t out_is_f32;
    int32_t D;
    int32_t resident;         // host-side choice of the launch form; the kernels ignore it
    const int32_t *order;     // the row that takes the place of absolute row r (rows of like length side by side for the
                              // several-rows-per-warp kernels; aggregation-node rows that read the same neighbourhood
                              // side by side), or null for the rows as they are; the resident-warp kernels ignore it
};

// Long rows (more than long_row entries) are not walked by one warp: they are cut into segments that
// different warps sum into fp32 partial rows; whoever finishes a row's last segment adds them up.
// Passed to the kernels as a parameter of its own, and only to the instantiations that handle long
// rows: growing GatherArgs itself costs the plain row kernels registers.
struct SegArgs {
    int32_t long_row;
    int32_t seg_first;        // index (in the table) of this launch's first segment
    int32_t seg_count;        // segments of this launch
    const int4 *segs;         // this launch's segments: {row, first entry, end entry, slot of the row}
    const int2 *slots;        // per long row of the table: {index of its first segment, number of segments}
    unsigned int *seg_done;   // per long row: finished segments (zero between launches)
    float *partial;           // fp32 partial rows, indexed by the segment's index in its table
};

template <bool HAS_SEGS> struct KernelArgs { GatherArgs a; };
template <> struct KernelArgs<true> { GatherArgs a; SegArgs sg; };

template <typename T> struct Chunk;
template <> struct Chunk<float> { static constexpr int kElems = 4; };
template <> struct Chunk<__nv_bfloat16> { static constexpr int kElems = 8; };

// Programmatic dependent launch (PTX griddepcontrol).
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Feature rows and aggregation-node rows are read with ld.global.cg (coherent, cached at L2 only): the rows
// may have been written by the kernel before this one, which is still alive when this one starts under
// programmatic dependent launch, or by other warps of the same launch.  The non-coherent path
// (ld.global.nc, __ldg) is kept for the handle's static structure arrays only.
__device__ __forceinline__ float4 ld_f4(const void *p) { return __ldcg(reinterpret_cast<const float4 *>(p)); }
__device__ __forceinline__ uint4 ld_u4(const void *p) { return __ldcg(reinterpret_cast<const uint4 *>(p)); }

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

// a[0..E) += b[0..E) as packed fp32x2 adds (one instruction per two sums on sm_100; each half is an
// ordinary round-to-nearest add, so the bits are those of E scalar adds).
// Used for fp32 storage (4 sums per chunk); with 8 sums per chunk (bf16 storage) it was measured at every
// register budget from 40 to 64 and never beat scalar adds (spills at 40, too few warps above), so that
// path adds scalars.
template <int E>
__device__ __forceinline__ void add_rows(float *a, const float *b) {
    if constexpr (E == 4) {
#pragma unroll
        for (int j = 0; j < E; j += 2) {
            const float2 r = __fadd2_rn(make_float2(a[j], a[j + 1]), make_float2(b[j], b[j + 1]));
            a[j] = r.x;
            a[j + 1] = r.y;
        }
    } else {
#pragma unroll
        for (int j = 0; j < E; ++j) a[j] += b[j];
    }
}

// acc[0..8) += (factor *) the eight bf16 values of one 16-byte word group, widened two at a time (a bf16 is the
// upper half of an fp32: shift or mask) straight into packed fp32x2 adds: 8 widening and 4 arithmetic
// instructions per 16 bytes, and the raw words stay raw (4 registers, not 8) until they are used.
template <bool SCALED>
__device__ __forceinline__ void add_bf16x8(float *acc, const uint4 &r, float factor) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
    if constexpr (!SCALED) {
        // sm_100 adds a bf16 value to an fp32 one in one instruction (add.f32.bf16: the bf16 operand is widened exactly,
        // the sum rounded to nearest, i.e. the bits of widening first and adding then): 8 instructions per 16 bytes
        // instead of 8 shifts or masks and 4 packed adds
#pragma unroll
        for (int i = 0; i < 4; ++i)
            asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tadd.rn.f32.bf16 %0, lo, %0;\n\tadd.rn.f32.bf16 %1, hi, %1;\n\t}"
                : "+f"(acc[2 * i]), "+f"(acc[2 * i + 1])
                : "r"(w[i]));
    } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 x = make_float2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u));
        const float2 a = make_float2(acc[2 * i], acc[2 * i + 1]);
        const float2 s = SCALED ? __ffma2_rn(x, make_float2(factor, factor), a) : __fadd2_rn(a, x);
        acc[2 * i] = s.x;
        acc[2 * i + 1] = s.y;
    }
    }
}

// Per-lane view of the two source tables: byte pointers already offset to the
// lane's chunk, so a row address is one multiply-add.
template <typename T>
struct Tables {
    const char *prim;   // primary base + chunk offset
    const char *sec;    // secondary base + chunk offset - n_prim * sec_row_bytes
    int32_t n_prim;
    uint32_t prim_row_bytes, sec_row_bytes;
    __device__ __forceinline__ Tables(const void *p, const float *s, int32_t n, int32_t D, int chunk) {
        constexpr int E = Chunk<T>::kElems;
        n_prim = n;
        prim_row_bytes = uint32_t(D) * sizeof(T);
        sec_row_bytes = uint32_t(D) * 4u;
        prim = reinterpret_cast<const char *>(p) + size_t(chunk) * 16;
        // never dereferenced for ids < n_prim, so the wrapped offset is harmless when s is null
        sec = reinterpret_cast<const char *>(s) + size_t(chunk) * (E * 4) - size_t(n) * sec_row_bytes;
    }
    // One source row chunk -> kElems floats.
    __device__ __forceinline__ void load(int32_t id, float *v) const {
        constexpr int E = Chunk<T>::kElems;
        if constexpr (E == 4) {
            const bool is_prim = id < n_prim;
            const char *base = is_prim ? prim : sec;
            const float4 q = ld_f4(base + size_t(uint32_t(id)) * prim_row_bytes);   // both tables have 4 D bytes per row
            v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        } else {
            if (id < n_prim) {
                bf16x8_to_f32(ld_u4(prim + size_t(uint32_t(id)) * prim_row_bytes), v);
            } else {
                const char *p = sec + size_t(uint32_t(id)) * sec_row_bytes;
                const float4 q0 = ld_f4(p), q1 = ld_f4(p + 16);
                v[0] = q0.x; v[1] = q0.y; v[2] = q0.z; v[3] = q0.w;
                v[4] = q1.x; v[5] = q1.y; v[6] = q1.z; v[7] = q1.w;
            }
        }
    }
};

template <typename T>
__device__ __forceinline__ void store_chunk(void *out, int out_is_f32, int32_t D, int32_t out_row, int chunk, const float *v) {
    constexpr int E = Chunk<T>::kElems;
    if (out_is_f32) {
        float *p = reinterpret_cast<float *>(out) + size_t(out_row) * D + chunk * E;
#pragma unroll
        for (int i = 0; i < E; i += 4) *reinterpret_cast<float4 *>(p + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
    } else if constexpr (E == 4) {
        float *p = reinterpret_cast<float *>(out) + size_t(out_row) * D + chunk * 4;
        __stcs(reinterpret_cast<float4 *>(p), make_float4(v[0], v[1], v[2], v[3]));
    } else {
        __nv_bfloat16 *p = reinterpret_cast<__nv_bfloat16 *>(out) + size_t(out_row) * D + chunk * 8;
        __stcs(reinterpret_cast<uint4 *>(p), f32x8_to_bf16(v));
    }
}

// Where a finished row goes.  The kernels that write one kind of row build it from GatherArgs; the
// single-launch kernel chooses per row between the caller's output and the fp32 rows of the
// aggregation nodes.
struct RowOut {
    void *out;
    int32_t is_f32;
    int32_t row_offset;
};
__device__ __forceinline__ RowOut row_out_of(const GatherArgs &a) { return RowOut{a.out, a.out_is_f32 & 1, a.out_row_offset}; }
// How gather_row finds the output at the END of a row (nothing of it is kept in registers meanwhile).
struct OutOfArgs {       // the launch writes one kind of row: taken from GatherArgs
    static constexpr bool kMixed = false;
    __device__ __forceinline__ RowOut get(const GatherArgs &a, int32_t) const { return row_out_of(a); }
};
struct OutPartial {      // a segment's partial row
    static constexpr bool kMixed = false;
    float *partial;
    __device__ __forceinline__ RowOut get(const GatherArgs &, int32_t) const { return RowOut{partial, 1, 0}; }
};
struct OutByRow {        // single-launch kernel: aggregation-node rows (id >= n_prim) go to their fp32 rows
    static constexpr bool kMixed = true;
    float *ahat;
    __device__ __forceinline__ RowOut get(const GatherArgs &a, int32_t row) const {
        return row >= a.n_prim ? RowOut{ahat, 1, a.n_prim} : row_out_of(a);
    }
};

// A row of the single-launch kernel may read rows that other warps of the same launch write.  Its entries
// ascend, so the rows of the layer input come first and need nothing: the row is summed in two parts, the
// entries before the first such row at once, the rest after the warp has waited for the phase that writes
// the latest of them.  The wait sits between the two loops, never inside them.  NoGate: a single part.
struct NoGate {
    static constexpr bool kOn = false;
    __device__ __forceinline__ int32_t split(int32_t e) const { return e; }
    __device__ __forceinline__ void wait(int) const {}
};
struct FusedArgs;
__device__ __forceinline__ void fused_wait(const FusedArgs &k, int phase, int lane);
struct PhaseGate {
    static constexpr bool kOn = true;
    const FusedArgs *k;
    int32_t req;          // phase to wait for before the second part, -1: none, or known to be complete
    int32_t n_sec;        // entries of the second part (the last n_sec of the row)
    // (always cut at the same place, waiting or not: the order of the additions must not depend on timing)
    __device__ __forceinline__ int32_t split(int32_t e) const { return e - n_sec; }
    __device__ __forceinline__ void wait(int lane) const {
        if (req >= 0) fused_wait(*k, req, lane);
    }
};

// What a warp needs before it can start on a row: the first 32 source ids (one per
// lane, -1 past the end), their factors, and the row's own factor.  All of it is
// static structure, so it can be fetched while the previous row is still summed.
struct RowHead {
    int32_t id;
    float src_scale;
    float dst_scale;
};

template <bool SRC_SCALE>
__device__ __forceinline__ RowHead load_head(const GatherArgs &a, int32_t row, int32_t b, int32_t e, int lane) {
    RowHead h;
    h.id = (b + lane < e) ? __ldg(a.idx + b + lane) : -1;
    // the factor of each source travels with its id: fetched a batch ahead, handed round by shuffle
    h.src_scale = 1.0f;
    if constexpr (SRC_SCALE) h.src_scale = (h.id >= 0 && h.id < a.n_prim) ? __ldg(a.src_scale + h.id) : 1.0f;
    h.dst_scale = (a.dst_scale && row < a.n_prim) ? __ldg(a.dst_scale + row) : 1.0f;   // graph-node rows only
    return h;
}

// Gather-sum of one row [b, e) by one warp.  Returns with the result stored.
template <typename T, int LPR, int UNROLL, bool SRC_SCALE, bool SELF, typename Out = OutOfArgs, typename Gate = NoGate>
__device__ __forceinline__ void gather_row(const GatherArgs &a, const Out &osel, int32_t row, int32_t b, int32_t e, const RowHead &head, int lane,
                                           const Gate gate = Gate()) {
    constexpr int E = Chunk<T>::kElems;
    constexpr int G = 32 / LPR;                 // slices per warp
    constexpr int PER_BATCH = LPR;              // neighbours each slice takes from a batch of 32 ids
    constexpr int U = (UNROLL < PER_BATCH) ? UNROLL : PER_BATCH;
    const int slice = lane / LPR;
    const int gl = lane % LPR;
    const int n_chunks = a.D / E;
    const float dscale = head.dst_scale;
    const int32_t first = head.id;
    const float first_s = head.src_scale;

    for (int c0 = 0; c0 < n_chunks; c0 += LPR) {
        const int chunk = c0 + gl;
        const bool live = chunk < n_chunks;
        const Tables<T> tab(a.prim, a.sec, a.n_prim, a.D, live ? chunk : 0);
        // two-level sum: `part` collects the tree sums of one batch of 32 ids, `acc` the batches, so a row of n
        // terms passes through about n/32 + 32/U + log2(U) roundings instead of n/U
        float acc[E], part[E];
#pragma unroll
        for (int j = 0; j < E; ++j) acc[j] = 0.0f;

        int32_t mine = first;
        float mine_s = first_s;
        if (c0 != 0) {
            mine = (b + lane < e) ? __ldg(a.idx + b + lane) : -1;
            if constexpr (SRC_SCALE) mine_s = (mine >= 0 && mine < a.n_prim) ? __ldg(a.src_scale + mine) : 1.0f;
        }
        int32_t lo = b, hi = gate.split(e);
#pragma unroll 1
        for (int half = 0; half < (Gate::kOn ? 2 : 1); ++half) {
        if (Gate::kOn && half == 1) {           // the rows written by earlier phases, at the end of the row
            lo = hi;
            hi = e;
            if (lo >= hi) break;
            mine = (lo + lane < hi) ? __ldg(a.idx + lo + lane) : -1;     // ids are static: in flight during the wait
            mine_s = 1.0f;
            gate.wait(lane);
        }
        for (int32_t base = lo; base < hi; base += 32) {
            // first part: entries beyond it belong to the second part and must not be loaded yet
            const int32_t cur = (Gate::kOn && base + lane >= hi) ? -1 : mine;
            const float cur_s = mine_s;
            const int32_t nb = base + 32;
            mine = (nb + lane < hi) ? __ldg(a.idx + nb + lane) : -1;     // next batch of ids, in flight early
            if constexpr (SRC_SCALE) mine_s = (mine >= 0 && mine < a.n_prim) ? __ldg(a.src_scale + mine) : 1.0f;
            const int cnt = min(32, hi - base);
            if constexpr (E == 8) {
                // bf16 storage.  The ids of a row ascend, so the rows of the layer input (bf16) are the first n_p
                // entries of the batch and the fp32 rows of aggregation nodes the rest: two loops, neither of which
                // has to choose a table per entry.  bf16 rows are fetched as raw words, U in flight, and widened
                // only as they are added (add_bf16x8); sums go straight into the accumulator (the result is rounded
                // to 8 bits anyway).
                const int n_p = __popc(__ballot_sync(0xffffffffu, cur >= 0 && cur < a.n_prim));
#pragma unroll
                for (int k = 0; k < PER_BATCH; k += U) {
                    if (k * G < n_p) {
                        uint4 raw[U];
                        if ((k + U) * G <= n_p) {       // every entry of this group exists: no checks, no zero fill
#pragma unroll
                            for (int u = 0; u < U; ++u)
                                raw[u] = ld_u4(tab.prim + size_t(uint32_t(__shfl_sync(0xffffffffu, cur, (k + u) * G + slice))) * tab.prim_row_bytes);
                        } else {
#pragma unroll
                            for (int u = 0; u < U; ++u) {
                                const int32_t id = __shfl_sync(0xffffffffu, cur, (k + u) * G + slice);
                                raw[u] = ((k + u) * G + slice < n_p && live) ? ld_u4(tab.prim + size_t(uint32_t(id)) * tab.prim_row_bytes)
                                                                             : make_uint4(0u, 0u, 0u, 0u);
                            }
                        }
#pragma unroll
                        for (int u = 0; u < U; ++u) {
                            float sc = 1.0f;
                            if constexpr (SRC_SCALE) sc = __shfl_sync(0xffffffffu, cur_s, (k + u) * G + slice);
                            add_bf16x8<SRC_SCALE>(acc, raw[u], sc);
                        }
                    }
                }
                // the fp32 rows (never scaled): 32 bytes per lane and row, so half as many rows in flight for the same registers
                constexpr int US = (U >= 2) ? U / 2 : 1;
                for (int j0 = n_p; j0 < cnt; j0 += US * G) {
                    float4 q[US][2];
#pragma unroll
                    for (int u = 0; u < US; ++u) {
                        const int j = j0 + u * G + slice;
                        const int32_t id = __shfl_sync(0xffffffffu, cur, j < cnt ? j : 0);
                        if (j < cnt && live) {
                            const char *p = tab.sec + size_t(uint32_t(id)) * tab.sec_row_bytes;
                            q[u][0] = ld_f4(p);
                            q[u][1] = ld_f4(p + 16);
                        } else {
                            q[u][0] = q[u][1] = make_float4(0.f, 0.f, 0.f, 0.f);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < US; ++u) {
                        float2 s;
                        s = __fadd2_rn(make_float2(acc[0], acc[1]), make_float2(q[u][0].x, q[u][0].y)); acc[0] = s.x; acc[1] = s.y;
                        s = __fadd2_rn(make_float2(acc[2], acc[3]), make_float2(q[u][0].z, q[u][0].w)); acc[2] = s.x; acc[3] = s.y;
                        s = __fadd2_rn(make_float2(acc[4], acc[5]), make_float2(q[u][1].x, q[u][1].y)); acc[4] = s.x; acc[5] = s.y;
                        s = __fadd2_rn(make_float2(acc[6], acc[7]), make_float2(q[u][1].z, q[u][1].w)); acc[6] = s.x; acc[7] = s.y;
                    }
                }
            } else {
            if constexpr (E == 4) {       // fp32 storage: two-level sums
#pragma unroll
                for (int j = 0; j < E; ++j) part[j] = 0.0f;
            }
#pragma unroll
            for (int k = 0; k < PER_BATCH; k += U) {
                if (k * G < cnt) {
                    float v[U][E];
                    // Measured on B200: the unchecked path is 4-18 % faster for fp32 storage without per-source
                    // factors; with factors or bf16 storage the doubled loop body spills and loses 5-13 %.
                    constexpr bool kFastGroups = (E == 4) && !SRC_SCALE;
                    if (kFastGroups && (k + U) * G <= cnt) {
                        // every entry of this group exists: no checks, no zero fill (lanes beyond the row
                        // width read chunk 0 of a valid row and are never stored)
#pragma unroll
                        for (int u = 0; u < U; ++u) tab.load(__shfl_sync(0xffffffffu, cur, (k + u) * G + slice), v[u]);
                    } else {
#pragma unroll
                        for (int u = 0; u < U; ++u) {
                            const int32_t id = __shfl_sync(0xffffffffu, cur, (k + u) * G + slice);
                            if (id >= 0 && (kFastGroups || live)) {
                                tab.load(id, v[u]);
                            } else {
#pragma unroll
                                for (int j = 0; j < E; ++j) v[u][j] = 0.0f;
                            }
                        }
                    }
                    if constexpr (SRC_SCALE && E == 4) {
                        // part += factor * row as packed fused multiply-adds (fma.rn.f32x2): two instructions per
                        // loaded row instead of four multiplies and the adds of the tree
#pragma unroll
                        for (int u = 0; u < U; ++u) {
                            const float sc = __shfl_sync(0xffffffffu, cur_s, (k + u) * G + slice);
                            const float2 s2 = make_float2(sc, sc);
                            const float2 lo = __ffma2_rn(make_float2(v[u][0], v[u][1]), s2, make_float2(part[0], part[1]));
                            const float2 hi = __ffma2_rn(make_float2(v[u][2], v[u][3]), s2, make_float2(part[2], part[3]));
                            part[0] = lo.x; part[1] = lo.y; part[2] = hi.x; part[3] = hi.y;
                        }
                    } else {
                        if constexpr (SRC_SCALE) {
#pragma unroll
                            for (int u = 0; u < U; ++u) {
                                const float sc = __shfl_sync(0xffffffffu, cur_s, (k + u) * G + slice);
#pragma unroll
                                for (int j = 0; j < E; ++j) v[u][j] *= sc;
                            }
                        }
                        // balanced tree over the U loaded rows, then one add into the accumulator
#pragma unroll
                        for (int w = U / 2; w >= 1; w /= 2)
#pragma unroll
                            for (int u = 0; u < w; ++u) add_rows<E>(v[u], v[u + w]);
                        if constexpr (E == 4) add_rows<E>(part, v[0]);
                        else add_rows<E>(acc, v[0]);
                    }
                }
            }
            if constexpr (E == 4) add_rows<E>(acc, part);
            }
        }
        }
        // combine the slices (fixed butterfly), then slice 0 stores
#pragma unroll
        for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
            for (int j = 0; j < E; ++j) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], off);
        if (live && slice == 0) {
            if constexpr (SELF) {         // GCN: the row's own term, compiled only into the variants that need it
                if (!Out::kMixed || row < a.n_prim) {    // (the single-launch kernel also writes aggregation-node rows)
                    float self[E];
                    tab.load(row, self);
                    float sc = 1.0f;
                    if constexpr (SRC_SCALE) sc = __ldg(a.src_scale + row);
#pragma unroll
                    for (int j = 0; j < E; ++j) acc[j] = fmaf(self[j], sc, acc[j]);
                }
            }
#pragma unroll
            for (int j = 0; j < E; ++j) acc[j] *= dscale;
            const RowOut ro = osel.get(a, row);
            store_chunk<T>(ro.out, ro.is_f32, a.D, row - ro.row_offset, chunk, acc);
        }
    }
}

// One segment of a long row: partial sum into a.partial, then, if this was the row's last open
// segment, the fixed-order sum of all its partials into the output.  The completion count is an
// integer atomic; the order of the floating-point additions never depends on who finishes when.
template <typename T, int LPR, int UNROLL, bool SRC_SCALE, bool SELF>
__device__ __forceinline__ void gather_segment(const GatherArgs &a, const SegArgs &sa, int32_t seg_local, int lane) {
    constexpr int E = Chunk<T>::kElems;
    const int4 sg = __ldg(sa.segs + seg_local);
    const int32_t row = sg.x, b = sg.y, e = sg.z, slot = sg.w;
    RowHead head = load_head<SRC_SCALE>(a, row, b, e, lane);
    head.dst_scale = 1.0f;
    gather_row<T, LPR, UNROLL, SRC_SCALE, false, OutPartial>(a, OutPartial{sa.partial}, sa.seg_first + seg_local, b, e, head, lane);
    __threadfence();                                   // partial row visible before the count moves
    __syncwarp();
    const int2 sl = __ldg(sa.slots + slot);
    unsigned done = 0;
    if (lane == 0) done = atomicAdd(sa.seg_done + slot, 1u);
    done = __shfl_sync(0xffffffffu, done, 0);
    if (done != unsigned(sl.y) - 1u) return;
    __threadfence();
    if (lane == 0) sa.seg_done[slot] = 0;              // ready for the next launch
    const float dscale = (a.dst_scale && row < a.n_prim) ? __ldg(a.dst_scale + row) : 1.0f;
    const int n_chunks = a.D / E;
    for (int chunk = lane; chunk < n_chunks; chunk += 32) {
        float acc[E];
#pragma unroll
        for (int j = 0; j < E; ++j) acc[j] = 0.0f;
        for (int k = 0; k < sl.y; ++k) {
            const float *p = sa.partial + size_t(sl.x + k) * a.D + chunk * E;
#pragma unroll
            for (int j = 0; j < E; j += 4) {
                const float4 q = __ldcg(reinterpret_cast<const float4 *>(p + j));   // written by other SMs: read at L2
                acc[j] += q.x; acc[j + 1] += q.y; acc[j + 2] += q.z; acc[j + 3] += q.w;
            }
        }
        if constexpr (SELF) {
            {
                const Tables<T> tab(a.prim, a.sec, a.n_prim, a.D, chunk);
                float self[E];
                tab.load(row, self);
                float sc = 1.0f;
                if constexpr (SRC_SCALE) sc = __ldg(a.src_scale + row);
#pragma unroll
                for (int j = 0; j < E; ++j) acc[j] = fmaf(self[j], sc, acc[j]);
            }
        }
#pragma unroll
        for (int j = 0; j < E; ++j) acc[j] *= dscale;
        store_chunk<T>(a.out, a.out_is_f32 & 1, a.D, row - a.out_row_offset, chunk, acc);
    }
}

// Out of line on purpose: the row path of the kernels keeps its registers and code.
template <typename T, int LPR, int UNROLL, bool SRC_SCALE, bool SELF>
__device__ __noinline__ void gather_segment_call(const GatherArgs &a, const SegArgs &sa, int32_t seg_local, int lane) {
    gather_segment<T, LPR, UNROLL, SRC_SCALE, SELF>(a, sa, seg_local, lane);
}

// out[row] = (dst_scale[row]) * sum_{e in row} (src_scale[id_e]) * table[id_e]
// One warp per work item, one item per launched warp.  HAS_SEGS: the launch has long rows; their
// segments are the first items, and rows longer than a.long_row are left to them.  Without long
// rows the kernel is compiled without any of that.
template <typename T, int LPR, int UNROLL, bool SRC_SCALE, bool HAS_SEGS, bool SELF>
__device__ __forceinline__ void gather_sum_body(const KernelArgs<HAS_SEGS> &k) {
    const GatherArgs &a = k.a;
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    int r_local = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if constexpr (HAS_SEGS) {
        if (r_local < k.sg.seg_count) {
            pdl_wait();
            gather_segment_call<T, LPR, UNROLL, SRC_SCALE, SELF>(a, k.sg, r_local, lane);
            return;
        }
        r_local -= k.sg.seg_count;
    }
    if (r_local >= a.row_count) return;
    int32_t row = a.row_begin + r_local;
    if (a.order) row = __ldg(a.order + row);       // aggregation-node rows in the order of their neighbourhoods
    const int32_t b = __ldg(a.row_ptr + row), e = __ldg(a.row_ptr + row + 1);
    if constexpr (HAS_SEGS) {
        if (e - b > k.sg.long_row) return;
    }
    const RowHead head = load_head<SRC_SCALE>(a, row, b, e, lane);
    pdl_wait();        // structure arrays are static; features may come from the previous kernel
    gather_row<T, LPR, UNROLL, SRC_SCALE, SELF>(a, OutOfArgs{}, row, b, e, head, lane);
}

// Two entry points per form: the parameter block of the variant with long rows is declared
// __grid_constant__ (its address is handed to the out-of-line segment function without a local
// copy); the variant without long rows takes plain parameters, which costs it fewer registers.
template <typename T, int LPR, int UNROLL, bool SRC_SCALE, int MIN_BLOCKS, bool SELF>
__global__ void __launch_bounds__(kThreads, MIN_BLOCKS) gather_sum_kernel(const KernelArgs<false> k) {
    gather_sum_body<T, LPR, UNROLL, SRC_SCALE, false, SELF>(k);
}
template <typename T, int LPR, int UNROLL, bool SRC_SCALE, int MIN_BLOCKS, bool SELF>
__global__ void __launch_bounds__(kThreads, MIN_BLOCKS) gather_sum_long_kernel(const __grid_constant__ KernelArgs<true> k) {
    gather_sum_body<T, LPR, UNROLL, SRC_SCALE, true, SELF>(k);
}

// Several rows per warp, for rows of 256 bytes or less (LPR < 32).  gather_row spreads ONE row over the warp's
// 32 / LPR lane groups and adds the groups' sums up at the end; with the short rows of clustered graphs (half of them
// 8 entries or fewer once a HAG has taken their common pairs away) most of the ~150 instructions around the loads
// are spent per row, not per entry, and the kernel is bound by instruction issue.  Here every lane group takes a row
// of its own: G = 32 / LPR rows share each instruction, no sums cross lanes, and a group keeps U loads of its row in
// flight.  The groups of a warp run in lock step for as long as the longest of their rows lasts.
// Order of additions of a row: per batch of LPR ids the tree sums of U rows at a time into `part`, batches into the
// accumulator (two-level, as in gather_row).
template <typename T, int LPR, int UNROLL, bool SRC_SCALE, bool HAS_SEGS, bool SELF, int ITEMS>
__device__ __forceinline__ void gather_sum_sub_body(const KernelArgs<HAS_SEGS> &k) {
    static_assert(LPR < 32, "one row per warp is gather_row's job");
    const GatherArgs &a = k.a;
    pdl_launch_dependents();
    constexpr int E = Chunk<T>::kElems;
    constexpr int G = 32 / LPR;
    constexpr int U = (UNROLL < LPR) ? UNROLL : LPR;
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    int item = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if constexpr (HAS_SEGS) {
        if (item < k.sg.seg_count) {
            pdl_wait();
            gather_segment_call<T, LPR, UNROLL, SRC_SCALE, SELF>(a, k.sg, item, lane);
            return;
        }
        item -= k.sg.seg_count;
    }
    const int slice = lane / LPR, gl = lane % LPR;
    // ITEMS groups of G rows per warp, one after the other: their row numbers, pointers and first ids are fetched
    // together, so the order -> pointers -> ids chain of latencies is paid once per warp, not once per group.
    // Measured on B200 with two groups: -3 % on 500 000 rows (cfg 4), +12 % and +36 % on 100 000 and 50 000 rows
    // (half as many warps to fill the machine with): the host asks for two only on the largest launches.
    item *= ITEMS;
    if (item * G >= a.row_count) return;
    bool have_[ITEMS];
    int32_t row_[ITEMS], b_[ITEMS], e_[ITEMS], mine_[ITEMS];
    float mine_s_[ITEMS], dscale_[ITEMS];
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        const int32_t r_local = (item + i) * G + slice;
        have_[i] = r_local < a.row_count;
        row_[i] = a.row_begin + (have_[i] ? r_local : 0);
    }
    if (a.order) {
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) row_[i] = __ldg(a.order + row_[i]);
    }
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        b_[i] = e_[i] = 0;
        if (have_[i]) {
            b_[i] = __ldg(a.row_ptr + row_[i]);
            e_[i] = __ldg(a.row_ptr + row_[i] + 1);
        }
    }
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        if constexpr (HAS_SEGS) {
            if (e_[i] - b_[i] > k.sg.long_row) { have_[i] = false; e_[i] = b_[i]; }      // a long row: its segments are items of their own
        }
        mine_[i] = (b_[i] + gl < e_[i]) ? __ldg(a.idx + b_[i] + gl) : -1;
        mine_s_[i] = 1.0f;
        if constexpr (SRC_SCALE) mine_s_[i] = (mine_[i] >= 0 && mine_[i] < a.n_prim) ? __ldg(a.src_scale + mine_[i]) : 1.0f;
        dscale_[i] = (have_[i] && a.dst_scale && row_[i] < a.n_prim) ? __ldg(a.dst_scale + row_[i]) : 1.0f;
    }
    pdl_wait();        // structure arrays are static; features may come from the previous kernel
    static_assert(ITEMS == 1 || ITEMS == 2, "the loop below selects between two sets of registers");
#pragma unroll 1        // one copy of the loop body: two would not fit the register budget
    for (int it = 0; it < ITEMS; ++it) {
    if ((item + it) * G >= a.row_count) break;
    const bool have = it ? have_[ITEMS - 1] : have_[0];
    const int32_t row = it ? row_[ITEMS - 1] : row_[0], b = it ? b_[ITEMS - 1] : b_[0], e = it ? e_[ITEMS - 1] : e_[0];
    int32_t mine = it ? mine_[ITEMS - 1] : mine_[0];
    float mine_s = it ? mine_s_[ITEMS - 1] : mine_s_[0];
    const float dscale = it ? dscale_[ITEMS - 1] : dscale_[0];
    const int32_t len = e - b;
    const int32_t max_len = __reduce_max_sync(FULL, len);
    const int n_chunks = a.D / E;
    const bool live = gl < n_chunks;
    const Tables<T> tab(a.prim, a.sec, a.n_prim, a.D, live ? gl : 0);
    float acc[E];
#pragma unroll
    for (int j = 0; j < E; ++j) acc[j] = 0.0f;
    for (int32_t off = 0; off < max_len; off += LPR) {
        const int32_t cur = mine;
        const float cur_s = mine_s;
        const int32_t nb = b + off + LPR + gl;
        mine = (nb < e) ? __ldg(a.idx + nb) : -1;                 // next batch of ids, in flight early
        if constexpr (SRC_SCALE) mine_s = (mine >= 0 && mine < a.n_prim) ? __ldg(a.src_scale + mine) : 1.0f;
        const int32_t cnt = len - off;                            // entries left in this group's row (<= 0: none)
        const int32_t max_cnt = max_len - off;
        float part[E];
#pragma unroll
        for (int j = 0; j < E; ++j) part[j] = 0.0f;
#pragma unroll
        for (int kk = 0; kk < LPR; kk += U) {
            if (kk < max_cnt) {
                float v[U][E];
                if (__all_sync(FULL, kk + U <= cnt)) {            // every group has U entries left: no checks, no fill
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
                            for (int j = 0; j < E; ++j) v[u][j] = 0.0f;
                        }
                    }
                }
                if constexpr (SRC_SCALE && E == 4) {
                    // part += factor * row as packed fused multiply-adds, as in gather_row
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const float sc = __shfl_sync(FULL, cur_s, kk + u, LPR);
                        const float2 s2 = make_float2(sc, sc);
                        const float2 lo = __ffma2_rn(make_float2(v[u][0], v[u][1]), s2, make_float2(part[0], part[1]));
                        const float2 hi = __ffma2_rn(make_float2(v[u][2], v[u][3]), s2, make_float2(part[2], part[3]));
                        part[0] = lo.x; part[1] = lo.y; part[2] = hi.x; part[3] = hi.y;
                    }
                } else {
                    if constexpr (SRC_SCALE) {
#pragma unroll
                        for (int u = 0; u < U; ++u) {
                            const float sc = __shfl_sync(FULL, cur_s, kk + u, LPR);
#pragma unroll
                            for (int j = 0; j < E; ++j) v[u][j] *= sc;
                        }
                    }
#pragma unroll
                    for (int w = U / 2; w >= 1; w /= 2)
#pragma unroll
                        for (int u = 0; u < w; ++u) add_rows<E>(v[u], v[u + w]);
                    add_rows<E>(part, v[0]);
                }
            }
        }
        add_rows<E>(acc, part);
    }
    if (have && live) {
        if constexpr (SELF) {         // GCN: the row's own term
            float self[E];
            tab.load(row, self);
            float sc = 1.0f;
            if constexpr (SRC_SCALE) sc = __ldg(a.src_scale + row);
#pragma unroll
            for (int j = 0; j < E; ++j) acc[j] = fmaf(self[j], sc, acc[j]);
        }
#pragma unroll
        for (int j = 0; j < E; ++j) acc[j] *= dscale;
        store_chunk<T>(a.out, a.out_is_f32 & 1, a.D, row - a.out_row_offset, gl, acc);
    }
    }
}

template <typename T, int LPR, int UNROLL, bool SRC_SCALE, int MIN_BLOCKS, bool SELF, int ITEMS>
__global__ void __launch_bounds__(kThreads, MIN_BLOCKS) gather_sum_sub_kernel(const KernelArgs<false> k) {
    gather_sum_sub_body<T, LPR, UNROLL, SRC_SCALE, false, SELF, ITEMS>(k);
}
template <typename T, int LPR, int UNROLL, bool SRC_SCALE, int MIN_BLOCKS, bool SELF, int ITEMS>
__global__ void __launch_bounds__(kThreads, MIN_BLOCKS) gather_sum_sub_long_kernel(const __grid_constant__ KernelArgs<true> k) {
    gather_sum_sub_body<T, LPR, UNROLL, SRC_SCALE, true, SELF, ITEMS>(k);
}

// The same, with resident warps that take items four at a time from a shared
// counter (a.sched[0]): first the segments of the long rows if there are any (the
// longest work goes first), then the rows, for which the next row's pointers and
// first ids are fetched while the current row is summed, so the pointer -> ids ->
// rows latency chain is paid once per warp instead of once per row.  The last warp
// to finish zeroes the counters (a.sched[1] counts finished warps) for the slot's
// next use.  No warp waits on another: there is no spin anywhere.
template <typename T, int LPR, int UNROLL, bool SRC_SCALE, bool HAS_SEGS, bool SELF>
__device__ __forceinline__ void gather_sum_persistent_body(const KernelArgs<HAS_SEGS> &k) {
    const GatherArgs &a = k.a;
    pdl_launch_dependents();
    constexpr int CH = 4;
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int32_t count = a.row_count;
    const int32_t *rp_base = a.row_ptr + a.row_begin;
    auto grab = [&]() -> int32_t {          // meaningful in lane 0
        int32_t v = 0;
        if (lane == 0) v = int32_t(atomicAdd(a.sched, unsigned(CH)));
        return v;
    };
    auto load_rp = [&](int32_t base) -> int32_t {   // lane i <= CH: pointer of row base + i (clamped to the end)
        return (lane <= CH && base < count) ? __ldg(rp_base + min(base + lane, count)) : 0;
    };
    int32_t seg_items = 0;
    int32_t base = __shfl_sync(FULL, grab(), 0);
    if constexpr (HAS_SEGS) {
        seg_items = (k.sg.seg_count + CH - 1) / CH * CH;    // segments occupy whole grabs
        pdl_wait();
        while (base < seg_items) {                          // each segment is long: no pipelining needed
#pragma unroll 1
            for (int i = 0; i < CH; ++i)
                if (base + i < k.sg.seg_count) gather_segment_call<T, LPR, UNROLL, SRC_SCALE, SELF>(a, k.sg, base + i, lane);
            base = __shfl_sync(FULL, grab(), 0);
        }
        base -= seg_items;
    }
    int32_t rp = load_rp(base);
    RowHead head{-1, 1.0f, 1.0f};
    if (base < count) head = load_head<SRC_SCALE>(a, a.row_begin + base, __shfl_sync(FULL, rp, 0), __shfl_sync(FULL, rp, 1), lane);
    if constexpr (!HAS_SEGS) pdl_wait();
    while (base < count) {
        const int32_t grabbed = grab();     // the next four rows; consumed after the first row below
        const int nrows = min(CH, count - base);
        int32_t nbase = count, rp_next = 0;
        for (int i = 0; i < nrows; ++i) {
            const int32_t b = __shfl_sync(FULL, rp, i), e = __shfl_sync(FULL, rp, i + 1);
            const RowHead cur = head;
            if (i + 1 < nrows) {
                head = load_head<SRC_SCALE>(a, a.row_begin + base + i + 1, e, __shfl_sync(FULL, rp, i + 2), lane);
            } else {
                if (nrows == 1) {
                    nbase = __shfl_sync(FULL, grabbed, 0) - seg_items;
                    rp_next = load_rp(nbase);
                }
                const int32_t nb = __shfl_sync(FULL, rp_next, 0), ne = __shfl_sync(FULL, rp_next, 1);
                if (nbase < count) head = load_head<SRC_SCALE>(a, a.row_begin + nbase, nb, ne, lane);
            }
            bool whole = true;
            if constexpr (HAS_SEGS) whole = e - b <= k.sg.long_row;
            if (whole) gather_row<T, LPR, UNROLL, SRC_SCALE, SELF>(a, OutOfArgs{}, a.row_begin + base + i, b, e, cur, lane);
            if (i == 0 && nrows > 1) {
                nbase = __shfl_sync(FULL, grabbed, 0) - seg_items;
                rp_next = load_rp(nbase);
            }
        }
        base = nbase;
        rp = rp_next;
    }
    if (lane == 0) {
        const unsigned finished = atomicAdd(a.sched + 1, 1u);
        if (finished == gridDim.x * kWarps - 1) {   // every warp has made its last grab
            a.sched[0] = 0;
            a.sched[1] = 0;
        }
    }
}

template <typename T, int LPR, int UNROLL, bool SRC_SCALE, int MIN_BLOCKS, bool SELF>
__global__ void __launch_bounds__(kThreads, MIN_BLOCKS) gather_sum_persistent_kernel(const KernelArgs<false> k) {
    gather_sum_persistent_body<T, LPR, UNROLL, SRC_SCALE, false, SELF>(k);
}
template <typename T, int LPR, int UNROLL, bool SRC_SCALE, int MIN_BLOCKS, bool SELF>
__global__ void __launch_bounds__(kThreads, MIN_BLOCKS) gather_sum_persistent_long_kernel(const __grid_constant__ KernelArgs<true> k) {
    gather_sum_persistent_body<T, LPR, UNROLL, SRC_SCALE, true, SELF>(k);
}

// --------------------------------------------------------------------------- //
// One whole pass as ONE launch.
//
// Algorithm 2 asks for the aggregation nodes in an order in which every node comes after its
// inputs, then the graph nodes.  Launching a kernel per level keeps that order but pays a launch
// and a pipeline drain per level, which costs more than the levels themselves once they are small
// (hierarchies of 7 to 20 levels whose sizes fall off geometrically).  Here the pass is a list of
// rows in that order -- phase 0, phase 1, ..., the graph-node rows last -- and resident warps take
// rows from the list four at a time.  Everything is a row: an aggregation node of a level that is
// evaluated pair by pair is a row of two entries; a row too long for one warp is cut into chunk rows
// of a phase of their own, whose fp32 partial rows (kept behind the aggregation nodes' rows, ids from
// n_prim + |V_A| on) a last short row adds up.  A row that reads rows of an earlier phase first
// waits until that phase's count of finished rows is complete.  The wait cannot deadlock (whatever
// is waited for was handed out earlier, to a warp that is running) and is bounded all the same: after
// spin_limit polls the warp records the failure (device word for the other waiters, host-mapped
// word for the caller), stops waiting and carries on, so the launch always ends.
// --------------------------------------------------------------------------- //
constexpr int kCtlNext = 0, kCtlFinished = 1, kCtlError = 2, kCtlDone = 4;
constexpr int kFusedGrab = 4;      // rows per grab; a grab lies in one phase

struct FusedArgs {
    GatherArgs a;              // idx: the pass's id list; prim / sec / n_prim / scales / out as for the row kernels;
                               // rows with id >= n_prim (aggregation nodes, chunk rows) go to ahat (fp32), row id - n_prim
    const int4 *items;         // {b, e, row, (required phase + 1) | phase << 8 | (entries read after the wait) << 16}; row < 0: padding
    int32_t n_items;           // a multiple of four; every group of four lies in one phase
    int32_t last_phase;        // its rows are not counted: nothing waits for them
    const int32_t *phase_size; // rows per phase, padding included
    unsigned int *ctl;         // [kCtlNext] next row, [kCtlFinished] finished warps, [kCtlError], [kCtlDone + p] finished rows of phase p
    float *ahat;               // = a.sec
    unsigned int *err_host;    // mapped host word, set when a wait ran out
    int32_t spin_limit;
    int32_t static_order;      // 0: warps take the next four rows from the shared counter (balances a long last phase);
                               // 1: warp w takes rows 4 w .. 4 w + 3, then the four W warps further on, and so on: no
                               // shared counter, for lists of many short phases, where one atomic per row on a single
                               // address costs more than the rows.  Needs every warp of the grid resident (as the
                               // launch guarantees: no more CTAs than fit), like any wait between warps.
};

// Every lane polls (one address: one request per poll) and the exits are taken on warp votes, so the
// control flow is uniform by construction: the code after the wait keeps plain converged shuffles.
__device__ __forceinline__ void fused_wait(const FusedArgs &k, int phase, int lane) {
    constexpr unsigned FULL = 0xffffffffu;
    const unsigned need = unsigned(__ldg(k.phase_size + phase));
    const unsigned int *done = k.ctl + kCtlDone + phase;
    const volatile unsigned int *failed = k.ctl + kCtlError;
    bool ok = false;
    for (int it = 0; it < k.spin_limit; ++it) {
        unsigned v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(done) : "memory");
        if (__all_sync(FULL, v >= need)) { ok = true; break; }
        if (__any_sync(FULL, *failed != 0u)) break;     // somebody gave up already: do not add a second of waiting per row
        // thousands of warps may wait for the same word, which is also the word the finishing warps add to: back off
        // quickly, so that the polls do not stand in the way of what they wait for
        __nanosleep(it < 2 ? 100 : (it < 6 ? 400 : 1000));
    }
    if (!ok && lane == 0) {
        k.ctl[kCtlError] = 1u;
        *reinterpret_cast<volatile unsigned int *>(k.err_host) = 1u;
        __threadfence_system();
    }
    __syncwarp();
    __threadfence();
}

template <typename T, int LPR, int UNROLL, bool SRC_SCALE, bool SELF>
__device__ __forceinline__ void fused_body(const FusedArgs &k) {
    const GatherArgs &a = k.a;
    pdl_launch_dependents();
    constexpr int CH = kFusedGrab;
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int32_t count = k.n_items;
    const int32_t stride = k.static_order ? int32_t(gridDim.x) * kWarps * CH : 0;
    int32_t next_static = (int32_t(blockIdx.x) * kWarps + int32_t(threadIdx.x >> 5)) * CH;
    auto grab = [&]() -> int32_t {          // meaningful in lane 0
        int32_t v = next_static;
        if (stride) next_static = min(next_static + stride, count);      // (count: nothing left; never overflows)
        else if (lane == 0) v = int32_t(atomicAdd(k.ctl + kCtlNext, unsigned(CH)));
        return v;
    };
    // the four rows of a grab in ONE register per lane: lane 4 w + i holds word w (b, e, row, phases) of row i
    auto load_items = [&](int32_t at) -> int32_t {
        return (lane < 4 * CH && at < count) ? __ldg(reinterpret_cast<const int32_t *>(k.items) + 4 * (at + (lane & 3)) + (lane >> 2)) : -1;
    };
    // first ids (and factors) of a row; nothing for padding
    auto item_head = [&](int32_t words, int i) -> RowHead {
        const int32_t b = __shfl_sync(FULL, words, i), e = __shfl_sync(FULL, words, 4 + i), row = __shfl_sync(FULL, words, 8 + i);
        if (row >= 0) return load_head<SRC_SCALE>(a, row, b, e, lane);
        return RowHead{-1, 1.0f, 1.0f};
    };
    int32_t base = __shfl_sync(FULL, grab(), 0);
    int32_t it = load_items(base);
    RowHead head = item_head(it, 0);
    int known = -1;            // every phase <= known has been seen complete: no need to look again
    unsigned pending = 0;      // rows of the current phase this warp has finished and not yet reported
    pdl_wait();        // the row list is static; features may come from the kernel before
    while (base < count) {
        const int32_t grabbed = grab();     // the next four rows; consumed after the first row below
        int32_t nbase = count, nit = -1;
        const int phase = (__shfl_sync(FULL, it, 12) >> 8) & 255;
#pragma unroll 1
        for (int i = 0; i < CH; ++i) {
            const int32_t b = __shfl_sync(FULL, it, i), e = __shfl_sync(FULL, it, 4 + i);
            const int32_t row = __shfl_sync(FULL, it, 8 + i), word = __shfl_sync(FULL, it, 12 + i);
            const RowHead cur = head;
            head = (i + 1 < CH) ? item_head(it, i + 1) : item_head(nit, 0);
            if (row >= 0) {
                const int req = (word & 255) - 1;
                gather_row<T, LPR, UNROLL, SRC_SCALE, SELF, OutByRow, PhaseGate>(a, OutByRow{k.ahat}, row, b, e, cur, lane,
                                                                                 PhaseGate{&k, req > known ? req : -1, int32_t(uint32_t(word) >> 16)});
                known = max(known, req);        // the row has waited for it (a row that waits for a phase reads from it)
            }
            if (i == 0) {
                nbase = __shfl_sync(FULL, grabbed, 0);
                nit = load_items(nbase);
            }
        }
        pending += unsigned(CH);
        // Finished rows are reported when the warp leaves their phase: its next grab lies in a later phase, or there is
        // none (rows are handed out in list order, so that is the moment the phase runs out of rows to hand out).
        // Always BEFORE the warp can wait for anything in the later phase, or it would wait for itself.
        const int next_phase = nbase < count ? (__shfl_sync(FULL, nit, 12) >> 8) & 255 : -1;
        if (next_phase != phase) {
            if (phase != k.last_phase) {
                // Reported only once the phase before is complete, so that "phase q is complete" implies that every
                // earlier phase is (a row waits for the latest phase it reads from only).
                if (phase - 1 > known) {
                    fused_wait(k, phase - 1, lane);
                    known = phase - 1;
                }
                __threadfence();                // this warp's rows visible before the count moves
                __syncwarp();
                if (lane == 0) atomicAdd(k.ctl + kCtlDone + phase, pending);
            }
            pending = 0;
        }
        base = nbase;
        it = nit;
    }
    if (lane == 0) {
        const unsigned finished = atomicAdd(k.ctl + kCtlFinished, 1u);
        if (finished == gridDim.x * kWarps - 1) {   // every warp has made its last grab and finished its rows
            for (int p = 0; p <= k.last_phase; ++p) k.ctl[kCtlDone + p] = 0;
            k.ctl[kCtlNext] = 0;
            k.ctl[kCtlError] = 0;
            k.ctl[kCtlFinished] = 0;
        }
    }
}

template <typename T, int LPR, int UNROLL, bool SRC_SCALE, int MIN_BLOCKS, bool SELF>
__global__ void __launch_bounds__(kThreads, MIN_BLOCKS) fused_pass_kernel(const __grid_constant__ FusedArgs k) {
    fused_body<T, LPR, UNROLL, SRC_SCALE, SELF>(k);
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

// Nodes per lane group: their input pairs are fetched together and all their row loads are in
// flight before the first add, so a group pays the pointer -> rows latency once for kPairBatch nodes.
constexpr int kPairBatch = 4;

template <typename T, int LPR>
__global__ void __launch_bounds__(kThreads) pair_sum_kernel(const PairArgs p) {
    pdl_launch_dependents();
    constexpr int E = Chunk<T>::kElems;
    constexpr int GROUPS = 32 / LPR;
    const int lane = threadIdx.x & 31;
    const int gl = lane % LPR;
    const int64_t group = (int64_t(blockIdx.x) * kWarps + (threadIdx.x >> 5)) * GROUPS + lane / LPR;
    const int32_t j0 = int32_t(group * kPairBatch);
    if (j0 >= p.count) return;
    int2 in[kPairBatch];
#pragma unroll
    for (int t = 0; t < kPairBatch; ++t)
        in[t] = (j0 + t < p.count) ? __ldg(reinterpret_cast<const int2 *>(p.agg_in) + p.first + j0 + t) : make_int2(-1, -1);
    pdl_wait();
    const int n_chunks = p.D / E;
    for (int chunk = gl; chunk < n_chunks; chunk += LPR) {
        const Tables<T> tab(p.x, p.ahat, p.n, p.D, chunk);
        float u[kPairBatch][E], v[kPairBatch][E];
#pragma unroll
        for (int t = 0; t < kPairBatch; ++t) {
            if (in[t].x >= 0) {
                tab.load(in[t].x, u[t]);
                tab.load(in[t].y, v[t]);
            }
        }
#pragma unroll
        for (int t = 0; t < kPairBatch; ++t) {
            if (in[t].x >= 0) {
                float *o = p.ahat + size_t(p.first + j0 + t) * p.D + chunk * E;
#pragma unroll
                for (int i = 0; i < E; i += 4)
                    *reinterpret_cast<float4 *>(o + i) = make_float4(u[t][i] + v[t][i], u[t][i + 1] + v[t][i + 1],
                                                                     u[t][i + 2] + v[t][i + 2], u[t][i + 3] + v[t][i + 3]);
            }
        }
    }
}

}  // namespace hagk
