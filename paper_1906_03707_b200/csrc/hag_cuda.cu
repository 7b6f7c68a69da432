// Device side of the C ABI: upload of the structure arrays and the launch
// sequences of the forward / backward aggregation (Algorithm 2 and its adjoint).
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>      // header-only; a no-op unless a profiler is attached

#include <algorithm>
#include <cstdint>
#include <cstdlib>
#include <limits>
#include <new>
#include <utility>
#include <vector>

#include "hag_internal.h"
#include "hag_kernels.cuh"
#include "hag_launch.h"

namespace {

using hagl::aligned16;
using hagl::DeviceGuard;
using hagl::lanes_per_row;

template <typename V>
hag_status upload_i32(int32_t **dst, const V *src, size_t count) {
    std::vector<int32_t> tmp;
    try {
        if (hag_alloc_should_fail(0)) throw std::bad_alloc();
        tmp.resize(std::max<size_t>(count, 1));
    } catch (const std::bad_alloc &) {
        return HAG_ERR_OOM_HOST;
    }
    for (size_t i = 0; i < count; ++i) tmp[i] = int32_t(src[i]);
    if (hag_alloc_should_fail(1)) return HAG_ERR_OOM_DEVICE;         // test hook: as if cudaMalloc had no memory left
    cudaError_t err = cudaMalloc(reinterpret_cast<void **>(dst), tmp.size() * sizeof(int32_t));
    if (err == cudaErrorMemoryAllocation) { cudaGetLastError(); return HAG_ERR_OOM_DEVICE; }
    if (err != cudaSuccess) { cudaGetLastError(); return HAG_ERR_CUDA; }
    if (cudaMemcpy(*dst, tmp.data(), tmp.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaGetLastError();
        return HAG_ERR_CUDA;
    }
    return HAG_OK;
}

void free_device(hag *h) {
    hag_device_arrays &d = h->d;
    for (cudaEvent_t ev : h->events) cudaEventDestroy(ev);
    h->events.clear();
    for (seg_set *set : {&h->seg_res, &h->seg_t, &h->seg_csr, &h->seg_csr_t, &h->seg_ftail, &h->seg_btail}) {
        if (set->d_order) cudaFree(set->d_order);
        set->d_order = nullptr;
    }
    for (seg_set *set : {&h->seg_res, &h->seg_t, &h->seg_csr, &h->seg_csr_t, &h->seg_ftail, &h->seg_btail})
    for (seg_table *t = set->g; t != set->g + kSegGrans; ++t) {
        if (t->d_segs) cudaFree(t->d_segs);
        if (t->d_slots) cudaFree(t->d_slots);
        if (t->d_done) cudaFree(t->d_done);
        t->d_segs = t->d_slots = nullptr;
        t->d_done = nullptr;
    }
    for (fused_table *t : {&h->fz_fwd, &h->fz_bwd, &h->fz_csr, &h->fz_csr_t})
        for (int32_t **p : {&t->d_items, &t->d_phase_size, &t->d_ids})
            if (*p) { cudaFree(*p); *p = nullptr; }
    if (d.err_host) cudaFreeHost(d.err_host);
    // these point into the id lists freed above
    d.res_idx = d.ftail_idx = d.t_idx = d.btail_idx = d.csr_idx = d.csr_t_idx = nullptr;
    if (d.copy_in_stream) {
        cudaStreamSynchronize(d.copy_in_stream);
        cudaStreamDestroy(d.copy_in_stream);
    }
    for (int i = 0; i < 2; ++i) {
        if (d.in_ready[i]) cudaEventDestroy(d.in_ready[i]);
        if (d.in_free[i]) cudaEventDestroy(d.in_free[i]);
    }
    void *ptrs[] = {d.agg_in, d.res_ptr, d.res_idx, d.t_ptr, d.t_idx, d.csr_ptr, d.csr_idx, d.csr_t_ptr,
                    d.csr_t_idx, d.inv_degree, d.inv_degree1, d.stage_in, d.stage_in2, d.stage_out, d.stage_ws,
                    d.ftail_ptr, d.ftail_idx, d.btail_ptr, d.btail_idx, d.sched, d.fused_ctl};
    for (void *p : ptrs)
        if (p) cudaFree(p);
    d = hag_device_arrays{};
}

template <typename Args>
cudaError_t launch_pdl(void (*kernel)(Args), unsigned grid, const Args &args, cudaStream_t s) {
    return hagl::launch_pdl(kernel, grid, unsigned(hagk::kThreads), args, s);
}

// Launch shape of the gather (loads in flight per lane, resident warps per SM,
// one row per launched warp or resident warps that pull rows), from sweeps on
// B200 over the five workload shapes:
//   fp32, large launch, 512-byte rows   : resident warps, 8 loads, 32 warps/SM
//   fp32, large launch, narrower rows   : resident warps, 4 loads, 32 warps/SM
//   fp32, small launch                  : one row per warp, 4 loads, 40 warps/SM (32 with per-source factors)
//   bf16                                : one row per warp, 2 loads, 48 warps/SM
// (large = at least 131072 rows or 4 Mi source entries)
// Resident warps hide the pointer -> ids latency of the next row behind the
// current one, which pays once there are many rows per warp; with few rows the
// hardware's own block scheduling balances better.
constexpr int32_t kManyRows = 131072;
constexpr int64_t kManyEdges = int64_t(4) << 20;

// Persistent form: exactly as many CTAs as stay resident, rows handed out through a.sched.
template <typename Kernel, typename Args>
cudaError_t launch_persistent(Kernel kernel, const Args &a, int64_t items, int sm_count, cudaStream_t s) {
    int per_sm = 0;
    cudaError_t err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, hagk::kThreads, 0);
    if (err != cudaSuccess) return err;
    const int64_t want = (items + hagk::kWarps - 1) / hagk::kWarps;
    const unsigned grid = unsigned(std::max<int64_t>(1, std::min<int64_t>(want, int64_t(per_sm) * sm_count)));
    return launch_pdl(kernel, grid, a, s);
}

template <bool SEGS>
hagk::KernelArgs<SEGS> pack_args(const hagk::GatherArgs &a, const hagk::SegArgs &sg) {
    hagk::KernelArgs<SEGS> k;
    k.a = a;
    if constexpr (SEGS) k.sg = sg;
    return k;
}

// The kernel entry for a shape: plain parameters without long rows, grid-constant ones with.
template <typename T, int LPR, int U, bool SS, int MINB, bool SEGS, bool SELF>
auto plain_kernel() {
    if constexpr (SEGS) return hagk::gather_sum_long_kernel<T, LPR, U, SS, MINB, SELF>;
    else return hagk::gather_sum_kernel<T, LPR, U, SS, MINB, SELF>;
}
template <typename T, int LPR, int U, bool SS, int MINB, bool SEGS, bool SELF>
auto resident_kernel() {
    if constexpr (SEGS) return hagk::gather_sum_persistent_long_kernel<T, LPR, U, SS, MINB, SELF>;
    else return hagk::gather_sum_persistent_kernel<T, LPR, U, SS, MINB, SELF>;
}

template <typename T, int LPR, int U, bool SS, int MINB, bool SEGS, bool SELF, int ITEMS>
auto sub_kernel() {
    if constexpr (SEGS) return hagk::gather_sum_sub_long_kernel<T, LPR, U, SS, MINB, SELF, ITEMS>;
    else return hagk::gather_sum_sub_kernel<T, LPR, U, SS, MINB, SELF, ITEMS>;
}
constexpr int64_t kSubTwoGroupsRows = 262144;     // launches of this many rows give a warp two groups of rows

// A launch that cannot give every resident warp a group of rows is bound by the latency of one row, which is shorter
// with the whole warp on it.
constexpr int64_t kSubMinWarps = 4096;
inline bool use_sub_rows(int lpr, int64_t rows) { return lpr < 32 && rows >= kSubMinWarps * (32 / lpr); }

template <typename T, int LPR, bool SS, bool SEGS, bool SELF>
cudaError_t launch_gather_shape(const hagk::GatherArgs &ga, const hagk::SegArgs &sg, int sm_count, cudaStream_t s) {
    const hagk::KernelArgs<SEGS> a = pack_args<SEGS>(ga, sg);
    const int64_t items = int64_t(ga.row_count) + (SEGS ? sg.seg_count : 0);
    const unsigned grid = unsigned((items + hagk::kWarps - 1) / hagk::kWarps);
    if constexpr (LPR < 32) {
        if (use_sub_rows(LPR, ga.row_count)) {
            constexpr int G = 32 / LPR;
            const int64_t groups = (int64_t(ga.row_count) + G - 1) / G;
            const int items = ga.row_count >= kSubTwoGroupsRows ? 2 : 1;
            const int64_t sub_items = (groups + items - 1) / items + (SEGS ? sg.seg_count : 0);
            const unsigned sub_grid = unsigned((sub_items + hagk::kWarps - 1) / hagk::kWarps);
            // sweep on B200 (loads in flight per lane x CTAs per SM; cfg 2 / cfg 4 / clique-union step in ms): 4 x 10: 0.118 /
            // 0.685 / 0.198; 8 x 8: 0.105 / 0.674 / 0.185; 8 x 9: 0.106 / 0.661 / 0.185; 16 x 5: 0.111 / 0.793 / 0.201;
            // 2 x 16: 0.150 / 0.680 / 0.234.  A group walks its row alone, so loads in flight count for more here than
            // in gather_row, where G groups share a row.
            if constexpr (sizeof(T) == 4) {
                if (items == 2) return launch_pdl(sub_kernel<T, LPR, 8, SS, SS ? 8 : 9, SEGS, SELF, 2>(), sub_grid, a, s);
                return launch_pdl(sub_kernel<T, LPR, 8, SS, SS ? 8 : 9, SEGS, SELF, 1>(), sub_grid, a, s);
            } else {
                if (items == 2) return launch_pdl(sub_kernel<T, LPR, 2, SS, 8, SEGS, SELF, 2>(), sub_grid, a, s);
                return launch_pdl(sub_kernel<T, LPR, 2, SS, 8, SEGS, SELF, 1>(), sub_grid, a, s);
            }
        }
    }
    if constexpr (sizeof(T) == 4) {
        if (ga.resident) {
            // 512-byte rows and wider: 16 loads in flight per lane x 5 CTAs per SM (sweep on B200, cfg 3 step in ms: 8 x 8 2.44,
            // 8 x 7 2.41, 16 x 4 2.39, 16 x 5 2.33, 16 x 6 2.48 (spills), 32 x 3 2.46, 4 x 12 2.71, no resident warps 2.82)
            if constexpr (LPR == 32) return launch_persistent(resident_kernel<T, LPR, 16, SS, 5, SEGS, SELF>(), a, items, sm_count, s);
            return launch_persistent(resident_kernel<T, LPR, 4, SS, 8, SEGS, SELF>(), a, items, sm_count, s);
        }
        // the variant with per-source factors needs the registers of 8 CTAs per SM, or it spills
        if constexpr (SS) return launch_pdl(plain_kernel<T, LPR, 4, SS, 8, SEGS, SELF>(), grid, a, s);
        return launch_pdl(plain_kernel<T, LPR, 4, SS, 10, SEGS, SELF>(), grid, a, s);
    } else {
        // bf16 rows are fetched as raw words and widened as they are added: four loads in flight fit the 40 registers of
        // 12 CTAs per SM (sweep on B200: 4 x 12 beats 2 x 12, 4 x 10, 8 x 8, 4 x 8 and resident warps)
        return launch_pdl(plain_kernel<T, LPR, 4, SS, 12, SEGS, SELF>(), grid, a, s);
    }
}

template <typename T, int LPR, bool SS>
cudaError_t launch_gather_lpr(const hagk::GatherArgs &a, const hagk::SegArgs &sg, int sm_count, cudaStream_t s) {
    if (a.out_is_f32 & 2)   // GCN's own-row term: its own instantiations, so the others stay as they are
        return sg.seg_count > 0 ? launch_gather_shape<T, LPR, SS, true, true>(a, sg, sm_count, s)
                                : launch_gather_shape<T, LPR, SS, false, true>(a, sg, sm_count, s);
    return sg.seg_count > 0 ? launch_gather_shape<T, LPR, SS, true, false>(a, sg, sm_count, s)
                            : launch_gather_shape<T, LPR, SS, false, false>(a, sg, sm_count, s);
}

template <typename T>
cudaError_t launch_gather(const hag *h, hagk::GatherArgs a, const seg_set &set, float *partial, int64_t edges,
                          int n_chunks, cudaStream_t s) {
    if (a.row_count <= 0) return cudaSuccess;
    a.resident = (a.row_count >= kManyRows || edges >= kManyEdges) ? 1 : 0;
    const int lpr = lanes_per_row(n_chunks);
    const bool sub = use_sub_rows(lpr, a.row_count);
    // a lane group walks its row alone: nothing longer than 256 entries stays whole there
    const int gran = sub ? std::min(seg_gran_for_rows(a.row_count), 1) : seg_gran_for_rows(a.row_count);
    // the row order: always for the several-rows-per-warp kernels; for the one-row-per-warp kernel on launches of
    // aggregation-node rows large enough for it to matter (the resident-warp kernels take consecutive rows)
    const bool near_rows = a.row_begin >= h->n && a.row_count >= kOrderNearRows && !(a.resident && sizeof(T) == 4);
    a.order = (set.d_order && (sub || near_rows)) ? set.d_order - set.order_first_row : nullptr;
    const seg_table &table = set.g[gran];
    hagk::SegArgs sg{};
    sg.long_row = kSegLongRow[gran];
    // the segments of this launch's long rows: a contiguous run of the table (segments are sorted by row)
    if (!table.segs.empty()) {
        const int64_t total = table.count();
        auto first_at_or_after = [&](int64_t row) {
            int64_t lo = 0, hi = total;
            while (lo < hi) {
                const int64_t mid = (lo + hi) / 2;
                if (table.segs[4 * mid] < row) lo = mid + 1; else hi = mid;
            }
            return lo;
        };
        const int64_t lo = first_at_or_after(a.row_begin), hi = first_at_or_after(int64_t(a.row_begin) + a.row_count);
        sg.segs = reinterpret_cast<const int4 *>(table.d_segs) + lo;
        sg.slots = reinterpret_cast<const int2 *>(table.d_slots);
        sg.seg_done = table.d_done;
        sg.partial = partial;
        sg.seg_first = int32_t(lo);
        sg.seg_count = int32_t(hi - lo);
    }
    hag *hm = const_cast<hag *>(h);
    a.sched = h->d.sched + 2 * (hm->sched_seq++ % kSchedSlots);
    const bool ss = a.src_scale != nullptr;
    switch (lpr) {
        case 4: return ss ? launch_gather_lpr<T, 4, true>(a, sg, h->sm_count, s) : launch_gather_lpr<T, 4, false>(a, sg, h->sm_count, s);
        case 8: return ss ? launch_gather_lpr<T, 8, true>(a, sg, h->sm_count, s) : launch_gather_lpr<T, 8, false>(a, sg, h->sm_count, s);
        case 16: return ss ? launch_gather_lpr<T, 16, true>(a, sg, h->sm_count, s) : launch_gather_lpr<T, 16, false>(a, sg, h->sm_count, s);
        default: return ss ? launch_gather_lpr<T, 32, true>(a, sg, h->sm_count, s) : launch_gather_lpr<T, 32, false>(a, sg, h->sm_count, s);
    }
}

template <typename T>
cudaError_t launch_pairs(const hagk::PairArgs &p, int n_chunks, cudaStream_t s) {
    if (p.count <= 0) return cudaSuccess;
    const int lpr = lanes_per_row(n_chunks);
    const int rows_per_cta = hagk::kWarps * (32 / lpr) * hagk::kPairBatch;
    const unsigned grid = unsigned((p.count + rows_per_cta - 1) / rows_per_cta);
    switch (lpr) {
        case 4: return launch_pdl(hagk::pair_sum_kernel<T, 4>, grid, p, s);
        case 8: return launch_pdl(hagk::pair_sum_kernel<T, 8>, grid, p, s);
        case 16: return launch_pdl(hagk::pair_sum_kernel<T, 16>, grid, p, s);
        default: return launch_pdl(hagk::pair_sum_kernel<T, 32>, grid, p, s);
    }
}

// One pass as one launch (fused_pass_kernel): exactly as many CTAs as stay resident.
template <typename T, int LPR, bool SS, bool SELF>
cudaError_t launch_fused_shape(const hagk::FusedArgs &k, int sm_count, cudaStream_t s) {
    const int64_t warps = (int64_t(k.n_items) + kFusedItemsPerGrab - 1) / kFusedItemsPerGrab;
    if constexpr (sizeof(T) == 4) {
        if constexpr (LPR == 32 && !SS) return launch_persistent(hagk::fused_pass_kernel<T, LPR, 8, SS, 8, SELF>, k, warps, sm_count, s);
        return launch_persistent(hagk::fused_pass_kernel<T, LPR, 4, SS, 8, SELF>, k, warps, sm_count, s);
    } else {
        return launch_persistent(hagk::fused_pass_kernel<T, LPR, 2, SS, 10, SELF>, k, warps, sm_count, s);
    }
}

template <typename T>
cudaError_t launch_fused(const hag *h, const fused_table &t, hagk::GatherArgs a, float *ahat, int n_chunks, cudaStream_t s,
                         bool head_only = false) {
    hagk::FusedArgs k{};
    a.idx = t.d_ids;
    a.row_ptr = nullptr;
    a.row_begin = 0;
    a.row_count = 0;
    a.sec = ahat;
    a.n_prim = h->n;           // ids from n on: aggregation nodes, then the chunk rows of this pass
    k.a = a;
    k.items = reinterpret_cast<const int4 *>(t.d_items);
    // head_only: the list ends where the graph-node rows begin; last_phase still names their phase, which is then never
    // reached, so every phase that runs is counted and can be waited for
    k.n_items = int32_t(head_only ? t.head_items : t.n_items());
    k.last_phase = t.last_phase;
    k.phase_size = t.d_phase_size;
    hag *hm = const_cast<hag *>(h);
    k.ctl = h->d.fused_ctl + size_t(kFusedCtlWords) * (hm->fused_seq++ % kFusedCtlSlots);
    k.ahat = ahat;
    k.err_host = h->d.err_dev;
    k.spin_limit = h->spin_limit;
    k.static_order = head_only ? 1 : 0;
    const int lpr = lanes_per_row(n_chunks);
    const bool ss = a.src_scale != nullptr, self = !head_only && (a.out_is_f32 & 2) != 0;
#define HAG_FUSED_CASE(L)                                                                                          \
    case L:                                                                                                        \
        if (ss) return self ? launch_fused_shape<T, L, true, true>(k, h->sm_count, s) : launch_fused_shape<T, L, true, false>(k, h->sm_count, s); \
        return self ? launch_fused_shape<T, L, false, true>(k, h->sm_count, s) : launch_fused_shape<T, L, false, false>(k, h->sm_count, s);
    switch (lpr) {
        HAG_FUSED_CASE(4)
        HAG_FUSED_CASE(8)
        HAG_FUSED_CASE(16)
        default:
        HAG_FUSED_CASE(32)
    }
#undef HAG_FUSED_CASE
}

// Brackets each launch with an event pair when profiling is on; always counts launches.
struct Recorder {
    hag *h;
    cudaStream_t s;
    bool failed = false;
    int open_ranges = 0;
    Recorder(const hag *h_, cudaStream_t s_) : h(const_cast<hag *>(h_)), s(s_) {
        h->notes.clear();
        h->last_launches = 0;
    }
    ~Recorder() {                      // a launch that failed left its range open
        while (open_ranges-- > 0) nvtxRangePop();
    }
    void begin(int32_t kind, int64_t rows, int64_t edges) {
        static const char *const names[4] = {"hag: level pair sums", "hag: gather over aggregation nodes",
                                             "hag: gather over graph nodes", "hag: whole pass in one launch"};
        nvtxRangePushA(names[kind & 3]);       // one range per launch, nested in the call's range
        ++open_ranges;
        if (h->profile) {
            const size_t i = h->notes.size();
            while (h->events.size() < 2 * (i + 1)) {
                cudaEvent_t ev;
                if (cudaEventCreate(&ev) != cudaSuccess) { cudaGetLastError(); failed = true; return; }
                h->events.push_back(ev);
            }
            if (cudaEventRecord(h->events[2 * i], s) != cudaSuccess) { cudaGetLastError(); failed = true; }
        }
        h->notes.push_back({kind, rows, edges});
    }
    void end() {
        if (h->profile && !failed) {
            const size_t i = h->notes.size() - 1;
            if (cudaEventRecord(h->events[2 * i + 1], s) != cudaSuccess) { cudaGetLastError(); failed = true; }
        }
        ++h->last_launches;
        nvtxRangePop();
        --open_ranges;
    }
};

hag_status check_call(const hag *h, hag_dtype dtype, int32_t D, const void *in, const void *out) {
    if (!h || !in || !out) return HAG_ERR_NULL;
    if (dtype != HAG_F32 && dtype != HAG_BF16) return HAG_ERR_DTYPE;
    if (D <= 0) return HAG_ERR_ARG;
    const size_t elem = dtype == HAG_F32 ? 4 : 2;
    if ((size_t(D) * elem) % 16 != 0 || !aligned16(in) || !aligned16(out)) return HAG_ERR_ALIGN;
    if (h->device < 0) return HAG_ERR_NOT_ON_DEVICE;
    if (in == out) return HAG_ERR_ARG;
    return HAG_OK;
}

// Aggregation nodes of the forward pass (Algorithm 2 lines 5-6): levels 1..fwd_cut
// level by level with the pair kernel, every deeper node in one gather launch
// from its expansion.  rec may be null (no bookkeeping).
template <typename T>
hag_status enqueue_fwd_agg(const hag *h, int32_t D, const void *x, float *ws, float *partial, cudaStream_t s, Recorder *rec) {
    const int n_chunks = D / hagk::Chunk<T>::kElems;
    const hag_device_arrays &d = h->d;
    for (int32_t l = 1; l <= h->fwd_cut; ++l) {
        hagk::PairArgs p{};
        p.agg_in = d.agg_in;
        p.first = int32_t(h->level_ptr[l - 1]);
        p.count = int32_t(h->level_ptr[l] - h->level_ptr[l - 1]);
        p.x = x;
        p.ahat = ws;
        p.n = h->n;
        p.D = D;
        if (p.count <= 0) continue;
        if (rec) rec->begin(0, p.count, 2 * int64_t(p.count));
        if (launch_pairs<T>(p, n_chunks, s) != cudaSuccess) return HAG_ERR_CUDA;
        if (rec) rec->end();
    }
    const int32_t j0 = int32_t(h->level_ptr[h->fwd_cut]);
    if (j0 < h->num_agg) {
        hagk::GatherArgs a{};
        a.row_ptr = d.ftail_ptr - (h->n + j0);     // indexed by absolute row id
        a.idx = d.ftail_idx;
        a.row_begin = h->n + j0;
        a.row_count = h->num_agg - j0;
        a.prim = x;
        a.sec = ws;
        a.n_prim = h->n;
        a.out = ws;
        a.out_row_offset = h->n;
        a.out_is_f32 = 1;
        a.D = D;
        if (rec) rec->begin(1, a.row_count, int64_t(h->ftail_idx.size()));
        if (launch_gather<T>(h, a, h->seg_ftail, partial, int64_t(h->ftail_idx.size()), n_chunks, s) != cudaSuccess) return HAG_ERR_CUDA;
        if (rec) rec->end();
    }
    return HAG_OK;
}

// Forward: aggregation nodes, then the gather over the graph nodes (lines 7-8).
template <typename T>
hag_status fwd_impl(const hag *h, bool use_hag, hag_reduce reduce, int32_t D, const void *x, void *out, void *ws,
                    cudaStream_t s, Recorder *rec) {
    const int n_chunks = D / hagk::Chunk<T>::kElems;
    const hag_device_arrays &d = h->d;
    hagk::GatherArgs a{};
    a.row_begin = 0;
    a.row_count = h->n;
    a.prim = x;
    a.dst_scale = (reduce == HAG_MEAN) ? d.inv_degree : (reduce == HAG_GCN ? d.inv_degree1 : nullptr);
    a.out_is_f32 = (reduce == HAG_GCN) ? 2 : 0;      // GCN: add the node's own row before normalising
    a.out = out;
    a.D = D;
    a.n_prim = std::numeric_limits<int32_t>::max();
    // workspace layout: rows of the aggregation nodes (HAG calls only), then the partial rows of long-row segments
    float *partial = static_cast<float *>(ws) + (use_hag ? size_t(h->num_agg) * D : 0);
    const fused_table &fz = use_hag ? h->fz_fwd : h->fz_csr;
    if (h->schedule == 1 && fz.ok) {       // the whole pass in one launch; the plain graph's chunk rows start at ws row 0
        if (rec) rec->begin(3, int64_t(h->n) + (use_hag ? h->num_agg : 0), use_hag ? h->e_hat : h->e);
        if (launch_fused<T>(h, fz, a, static_cast<float *>(ws), n_chunks, s) != cudaSuccess) return HAG_ERR_CUDA;
        if (rec) rec->end();
        return HAG_OK;
    }
    if (use_hag) {
        if (h->num_agg > 0) {
            if (h->schedule == 2 && fz.ok && fz.head_items > 0) {     // the aggregation nodes, all levels, in one launch
                if (rec) rec->begin(3, h->num_agg, h->e_hat - h->e_res);
                if (launch_fused<T>(h, fz, a, static_cast<float *>(ws), n_chunks, s, true) != cudaSuccess) return HAG_ERR_CUDA;
                if (rec) rec->end();
            } else {
                hag_status st = enqueue_fwd_agg<T>(h, D, x, static_cast<float *>(ws), partial, s, rec);
                if (st != HAG_OK) return st;
            }
            a.sec = static_cast<const float *>(ws);
            a.n_prim = h->n;
        }
        a.row_ptr = d.res_ptr;
        a.idx = d.res_idx;
    } else {
        a.row_ptr = d.csr_ptr;
        a.idx = d.csr_idx;
    }
    if (h->n > 0) {
        if (rec) rec->begin(2, h->n, use_hag ? h->e_res : h->e);
        if (launch_gather<T>(h, a, use_hag ? h->seg_res : h->seg_csr, partial, use_hag ? h->e_res : h->e, n_chunks, s) != cudaSuccess) return HAG_ERR_CUDA;
        if (rec) rec->end();
    }
    return HAG_OK;
}

// Backward: gather over the transposed structure.  Nodes deeper than bwd_cut take
// their gradient straight from the graph-node outputs that use them, in one
// launch; levels bwd_cut..1 follow from the last to the first (their gradient
// rows live in the workspace); then the graph nodes as sources.  A destination
// id < n stands for the output row of that graph node (scaled by 1/|N| for
// mean), an id >= n for an aggregation node.
template <typename T>
hag_status bwd_impl(const hag *h, bool use_hag, hag_reduce reduce, int32_t D, const void *g, void *gx, void *ws,
                    cudaStream_t s, Recorder *rec) {
    const int n_chunks = D / hagk::Chunk<T>::kElems;
    const hag_device_arrays &d = h->d;
    hagk::GatherArgs a{};
    a.prim = g;
    a.src_scale = (reduce == HAG_MEAN) ? d.inv_degree : (reduce == HAG_GCN ? d.inv_degree1 : nullptr);
    a.D = D;
    a.n_prim = std::numeric_limits<int32_t>::max();
    float *partial = static_cast<float *>(ws) + (use_hag ? size_t(h->num_agg) * D : 0);
    const fused_table &fz = use_hag ? h->fz_bwd : h->fz_csr_t;
    if (h->schedule == 1 && fz.ok) {       // the whole pass in one launch
        a.out = gx;
        a.out_is_f32 = (reduce == HAG_GCN) ? 2 : 0;
        if (rec) rec->begin(3, int64_t(h->n) + (use_hag ? h->num_agg : 0), use_hag ? h->e_hat : h->e);
        if (launch_fused<T>(h, fz, a, static_cast<float *>(ws), n_chunks, s) != cudaSuccess) return HAG_ERR_CUDA;
        if (rec) rec->end();
        return HAG_OK;
    }
    if (use_hag && h->num_agg > 0 && h->schedule == 2 && fz.ok && fz.head_items > 0) {
        // the aggregation nodes' gradients, the expanded ones and every level, in one launch
        if (rec) rec->begin(3, h->num_agg, h->e_hat - h->t_ptr[h->n]);
        if (launch_fused<T>(h, fz, a, static_cast<float *>(ws), n_chunks, s, true) != cudaSuccess) return HAG_ERR_CUDA;
        if (rec) rec->end();
        a.row_ptr = d.t_ptr;
        a.idx = d.t_idx;
        a.sec = static_cast<const float *>(ws);
        a.n_prim = h->n;
    } else if (use_hag && h->num_agg > 0) {
        const int32_t j0 = int32_t(h->level_ptr[h->bwd_cut]);
        if (j0 < h->num_agg) {
            hagk::GatherArgs t = a;              // all sources are graph-node outputs
            t.row_ptr = d.btail_ptr - (h->n + j0);
            t.idx = d.btail_idx;
            t.row_begin = h->n + j0;
            t.row_count = h->num_agg - j0;
            t.out = ws;
            t.out_row_offset = h->n;
            t.out_is_f32 = 1;
            if (rec) rec->begin(1, t.row_count, int64_t(h->btail_idx.size()));
            if (launch_gather<T>(h, t, h->seg_btail, partial, int64_t(h->btail_idx.size()), n_chunks, s) != cudaSuccess) return HAG_ERR_CUDA;
            if (rec) rec->end();
        }
        a.row_ptr = d.t_ptr;
        a.idx = d.t_idx;
        a.sec = static_cast<const float *>(ws);
        a.n_prim = h->n;
        for (int32_t l = h->bwd_cut; l >= 1; --l) {
            hagk::GatherArgs lv = a;
            lv.row_begin = h->n + int32_t(h->level_ptr[l - 1]);
            lv.row_count = int32_t(h->level_ptr[l] - h->level_ptr[l - 1]);
            lv.out = ws;
            lv.out_row_offset = h->n;
            lv.out_is_f32 = 1;
            if (lv.row_count <= 0) continue;
            const int64_t lv_edges = h->t_ptr[size_t(lv.row_begin) + lv.row_count] - h->t_ptr[lv.row_begin];
            if (rec) rec->begin(1, lv.row_count, lv_edges);
            if (launch_gather<T>(h, lv, h->seg_t, partial, lv_edges, n_chunks, s) != cudaSuccess) return HAG_ERR_CUDA;
            if (rec) rec->end();
        }
    } else if (use_hag) {
        a.row_ptr = d.t_ptr;
        a.idx = d.t_idx;
    } else {
        a.row_ptr = d.csr_t_ptr;
        a.idx = d.csr_t_idx;
    }
    a.row_begin = 0;
    a.row_count = h->n;
    a.out = gx;
    a.out_is_f32 = (reduce == HAG_GCN) ? 2 : 0;      // GCN: plus the node's own scaled gradient row
    if (h->n > 0) {
        if (rec) rec->begin(2, h->n, use_hag ? h->t_ptr[h->n] : h->e);
        if (launch_gather<T>(h, a, use_hag ? h->seg_t : h->seg_csr_t, partial, use_hag ? h->t_ptr[h->n] : h->e, n_chunks, s) != cudaSuccess) return HAG_ERR_CUDA;
        if (rec) rec->end();
    }
    return HAG_OK;
}

hag_status run(const hag *h, bool backward, bool use_hag, hag_reduce reduce, hag_dtype dtype, int32_t D, const void *in,
               void *out, void *ws, void *stream) {
    hag_status st = check_call(h, dtype, D, in, out);
    if (st != HAG_OK) return st;
    if (reduce != HAG_SUM && reduce != HAG_MEAN && reduce != HAG_GCN) return HAG_ERR_ARG;
    const bool needs_ws = use_hag ? (h->num_agg > 0 || h->max_segs_hag > 0) : (h->max_segs_csr > 0);
    if (needs_ws) {
        if (!ws) return HAG_ERR_WORKSPACE;
        if (!aligned16(ws)) return HAG_ERR_ALIGN;
    }
    DeviceGuard guard(h->device);
    if (!guard.ok) { cudaGetLastError(); return HAG_ERR_CUDA; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Recorder rec(h, s);
    nvtxRangePushA(use_hag ? (backward ? "hag_aggregate_bwd" : "hag_aggregate_fwd") : (backward ? "csr_aggregate_bwd" : "csr_aggregate_fwd"));
    if (dtype == HAG_F32)
        st = backward ? bwd_impl<float>(h, use_hag, reduce, D, in, out, ws, s, &rec)
                      : fwd_impl<float>(h, use_hag, reduce, D, in, out, ws, s, &rec);
    else
        st = backward ? bwd_impl<__nv_bfloat16>(h, use_hag, reduce, D, in, out, ws, s, &rec)
                      : fwd_impl<__nv_bfloat16>(h, use_hag, reduce, D, in, out, ws, s, &rec);
    nvtxRangePop();
    if (st == HAG_OK && rec.failed) st = HAG_ERR_CUDA;
    return st;
}

hag_status grow(void **buf, size_t *have, size_t need) {
    if (*have >= need) return HAG_OK;
    if (*buf) cudaFree(*buf);
    *buf = nullptr;
    *have = 0;
    cudaError_t err = cudaMalloc(buf, need);
    if (err == cudaErrorMemoryAllocation) { cudaGetLastError(); return HAG_ERR_OOM_DEVICE; }
    if (err != cudaSuccess) { cudaGetLastError(); return HAG_ERR_CUDA; }
    *have = need;
    return HAG_OK;
}

}  // namespace

extern "C" hag_status hag_destroy(hag_t *h) {
    if (!h) return HAG_OK;
    if (h->device >= 0) {
        DeviceGuard guard(h->device);
        if (guard.ok) free_device(h);
    }
    delete h;
    return HAG_OK;
}

extern "C" hag_status hag_to_device(hag_t *h, int device) {
    if (!h) return HAG_ERR_NULL;
    if (device < 0) return HAG_ERR_ARG;
    if (h->device == device) return HAG_OK;
    if (h->device >= 0) return HAG_ERR_ARG;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess) { cudaGetLastError(); return HAG_ERR_CUDA; }
    if (device >= count) return HAG_ERR_ARG;
    DeviceGuard guard(device);
    if (!guard.ok) { cudaGetLastError(); return HAG_ERR_CUDA; }
    hag_device_arrays &d = h->d;
    hag_status st = HAG_OK;
    const size_t n = size_t(h->n), k = size_t(h->num_agg);
    if (st == HAG_OK) st = upload_i32(&d.agg_in, h->agg_in.data(), 2 * k);
    if (st == HAG_OK) st = upload_i32(&d.res_ptr, h->res_ptr.data(), n + 1);
    // the id lists of the four passes: row lists and expansion lists are parts of them
    if (st == HAG_OK) st = upload_i32(&h->fz_fwd.d_ids, h->fz_fwd.ids.data(), h->fz_fwd.ids.size());
    if (st == HAG_OK) st = upload_i32(&h->fz_bwd.d_ids, h->fz_bwd.ids.data(), h->fz_bwd.ids.size());
    if (st == HAG_OK) st = upload_i32(&h->fz_csr.d_ids, h->fz_csr.ids.data(), h->fz_csr.ids.size());
    if (st == HAG_OK) st = upload_i32(&h->fz_csr_t.d_ids, h->fz_csr_t.ids.data(), h->fz_csr_t.ids.size());
    if (st == HAG_OK) {
        d.ftail_idx = h->fz_fwd.d_ids + h->fz_fwd.off_head;
        d.res_idx = h->fz_fwd.d_ids + h->fz_fwd.off_tail;
        d.btail_idx = h->fz_bwd.d_ids + h->fz_bwd.off_head;
        d.t_idx = h->fz_bwd.d_ids + h->fz_bwd.off_tail;
        d.csr_idx = h->fz_csr.d_ids + h->fz_csr.off_tail;
        d.csr_t_idx = h->fz_csr_t.d_ids + h->fz_csr_t.off_tail;
    }
    if (st == HAG_OK) st = upload_i32(&d.t_ptr, h->t_ptr.data(), n + k + 1);
    if (st == HAG_OK) st = upload_i32(&d.csr_ptr, h->csr_ptr.data(), n + 1);
    if (st == HAG_OK) st = upload_i32(&d.csr_t_ptr, h->csr_t_ptr.data(), n + 1);
    if (st == HAG_OK) st = upload_i32(&d.ftail_ptr, h->ftail_ptr.data(), h->ftail_ptr.size());
    if (st == HAG_OK) st = upload_i32(&d.btail_ptr, h->btail_ptr.data(), h->btail_ptr.size());
    if (st == HAG_OK) {
        std::vector<float> inv(std::max<size_t>(n, 1), 1.0f), inv1(std::max<size_t>(n, 1), 1.0f);
        for (size_t v = 0; v < n; ++v) {
            inv[v] = h->in_degree[v] > 0 ? 1.0f / float(h->in_degree[v]) : 1.0f;
            inv1[v] = 1.0f / float(h->in_degree[v] + 1);
        }
        for (auto pr : {std::make_pair(&d.inv_degree, &inv), std::make_pair(&d.inv_degree1, &inv1)}) {
            if (st != HAG_OK) break;
            cudaError_t err = cudaMalloc(reinterpret_cast<void **>(pr.first), pr.second->size() * sizeof(float));
            if (err != cudaSuccess) {
                cudaGetLastError();
                st = err == cudaErrorMemoryAllocation ? HAG_ERR_OOM_DEVICE : HAG_ERR_CUDA;
            } else if (cudaMemcpy(*pr.first, pr.second->data(), pr.second->size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) {
                cudaGetLastError();
                st = HAG_ERR_CUDA;
            }
        }
    }
    for (seg_set *set : {&h->seg_res, &h->seg_t, &h->seg_csr, &h->seg_csr_t, &h->seg_ftail, &h->seg_btail})
        if (st == HAG_OK && !set->order.empty()) st = upload_i32(&set->d_order, set->order.data(), set->order.size());
    for (seg_set *set : {&h->seg_res, &h->seg_t, &h->seg_csr, &h->seg_csr_t, &h->seg_ftail, &h->seg_btail})
    for (seg_table *t = set->g; t != set->g + kSegGrans; ++t) {
        if (st != HAG_OK || t->segs.empty()) continue;
        st = upload_i32(&t->d_segs, t->segs.data(), t->segs.size());
        if (st == HAG_OK) st = upload_i32(&t->d_slots, t->slots.data(), t->slots.size());
        if (st == HAG_OK) {
            const size_t bytes = (t->slots.size() / 2) * sizeof(unsigned int);
            if (cudaMalloc(reinterpret_cast<void **>(&t->d_done), bytes) != cudaSuccess || cudaMemset(t->d_done, 0, bytes) != cudaSuccess) {
                cudaGetLastError();
                st = HAG_ERR_CUDA;
            }
        }
    }
    if (st == HAG_OK) {
        const size_t bytes = size_t(2) * kSchedSlots * sizeof(unsigned int);
        if (cudaMalloc(reinterpret_cast<void **>(&d.sched), bytes) != cudaSuccess || cudaMemset(d.sched, 0, bytes) != cudaSuccess ||
            cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
            cudaGetLastError();
            st = HAG_ERR_CUDA;
        }
    }
    for (fused_table *t : {&h->fz_fwd, &h->fz_bwd, &h->fz_csr, &h->fz_csr_t}) {
        if (st != HAG_OK || !t->ok) continue;
        st = upload_i32(&t->d_items, t->items.data(), t->items.size());
        if (st == HAG_OK) st = upload_i32(&t->d_phase_size, t->phase_size.data(), t->phase_size.size());
    }
    if (st == HAG_OK) {
        const size_t bytes = size_t(kFusedCtlSlots) * kFusedCtlWords * sizeof(unsigned int);
        if (cudaMalloc(reinterpret_cast<void **>(&d.fused_ctl), bytes) != cudaSuccess || cudaMemset(d.fused_ctl, 0, bytes) != cudaSuccess ||
            cudaHostAlloc(reinterpret_cast<void **>(&d.err_host), sizeof(unsigned int), cudaHostAllocMapped) != cudaSuccess) {
            cudaGetLastError();
            st = HAG_ERR_CUDA;
        } else {
            *d.err_host = 0;
            if (cudaHostGetDevicePointer(reinterpret_cast<void **>(&d.err_dev), d.err_host, 0) != cudaSuccess) {
                cudaGetLastError();
                st = HAG_ERR_CUDA;
            }
        }
    }
    if (st != HAG_OK) {
        free_device(h);
        return st;
    }
    h->device = device;
    return HAG_OK;
}

extern "C" size_t hag_workspace_bytes(const hag_t *h, int32_t D) {
    if (!h || D <= 0) return 0;
    return (size_t(h->num_agg) + size_t(h->max_segs_hag)) * size_t(D) * sizeof(float);
}

extern "C" size_t csr_workspace_bytes(const hag_t *h, int32_t D) {
    if (!h || D <= 0) return 0;
    return size_t(h->max_segs_csr) * size_t(D) * sizeof(float);
}

extern "C" hag_status hag_aggregate_fwd(const hag_t *h, hag_reduce reduce, hag_dtype dtype, int32_t D, const void *x,
                                        void *out, void *workspace, void *cuda_stream) {
    return run(h, false, true, reduce, dtype, D, x, out, workspace, cuda_stream);
}

extern "C" hag_status hag_aggregate_bwd(const hag_t *h, hag_reduce reduce, hag_dtype dtype, int32_t D,
                                        const void *grad_out, void *grad_x, void *workspace, void *cuda_stream) {
    return run(h, true, true, reduce, dtype, D, grad_out, grad_x, workspace, cuda_stream);
}

extern "C" hag_status csr_aggregate_fwd(const hag_t *h, hag_reduce reduce, hag_dtype dtype, int32_t D, const void *x,
                                        void *out, void *workspace, void *cuda_stream) {
    return run(h, false, false, reduce, dtype, D, x, out, workspace, cuda_stream);
}

extern "C" hag_status csr_aggregate_bwd(const hag_t *h, hag_reduce reduce, hag_dtype dtype, int32_t D,
                                        const void *grad_out, void *grad_x, void *workspace, void *cuda_stream) {
    return run(h, true, false, reduce, dtype, D, grad_out, grad_x, workspace, cuda_stream);
}

extern "C" hag_status hag_aggregate_host(hag_t *h, int backward, int use_hag, hag_reduce reduce, hag_dtype dtype,
                                         int32_t D, const void *in_host, void *out_host, void *cuda_stream) {
    if (!h || !in_host || !out_host) return HAG_ERR_NULL;
    if (dtype != HAG_F32 && dtype != HAG_BF16) return HAG_ERR_DTYPE;
    if (D <= 0) return HAG_ERR_ARG;
    if (h->device < 0) return HAG_ERR_NOT_ON_DEVICE;
    const size_t bytes = size_t(h->n) * size_t(D) * (dtype == HAG_F32 ? 4 : 2);
    DeviceGuard guard(h->device);
    if (!guard.ok) { cudaGetLastError(); return HAG_ERR_CUDA; }
    hag_device_arrays &d = h->d;
    // Pipeline over consecutive calls: the copy-in runs on a stream of the handle's own into one of two input
    // buffers, so it overlaps the aggregation and the copy-out of the previous call (which stay on the caller's
    // stream, where the caller waits for the result).  Events order the reuse of the two buffers.
    if (!d.copy_in_stream) {
        if (cudaStreamCreateWithFlags(&d.copy_in_stream, cudaStreamNonBlocking) != cudaSuccess) { cudaGetLastError(); return HAG_ERR_CUDA; }
        for (int i = 0; i < 2; ++i) {
            if (cudaEventCreateWithFlags(&d.in_ready[i], cudaEventDisableTiming) != cudaSuccess ||
                cudaEventCreateWithFlags(&d.in_free[i], cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); return HAG_ERR_CUDA; }
        }
    }
    const uint32_t slot = d.host_calls & 1u;
    void **in_buf = slot ? &d.stage_in2 : &d.stage_in;
    size_t *in_have = slot ? &d.stage_in2_bytes : &d.stage_in_bytes;
    hag_status st = grow(in_buf, in_have, std::max<size_t>(bytes, 16));
    if (st == HAG_OK) st = grow(&d.stage_out, &d.stage_out_bytes, std::max<size_t>(bytes, 16));
    if (st == HAG_OK)
        st = grow(&d.stage_ws, &d.stage_ws_bytes, std::max<size_t>(std::max(hag_workspace_bytes(h, D), csr_workspace_bytes(h, D)), 16));
    if (st != HAG_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    bool ok = true;
    // the buffer is free once the aggregation of the call before last has read it
    if (d.host_calls >= 2) ok = ok && cudaStreamWaitEvent(d.copy_in_stream, d.in_free[slot], 0) == cudaSuccess;
    if (bytes) ok = ok && cudaMemcpyAsync(*in_buf, in_host, bytes, cudaMemcpyHostToDevice, d.copy_in_stream) == cudaSuccess;
    ok = ok && cudaEventRecord(d.in_ready[slot], d.copy_in_stream) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(s, d.in_ready[slot], 0) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return HAG_ERR_CUDA; }
    ++d.host_calls;
    st = run(h, backward != 0, use_hag != 0, reduce, dtype, D, *in_buf, d.stage_out, d.stage_ws, cuda_stream);
    if (st != HAG_OK) return st;
    if (cudaEventRecord(d.in_free[slot], s) != cudaSuccess) { cudaGetLastError(); return HAG_ERR_CUDA; }
    if (bytes && cudaMemcpyAsync(out_host, d.stage_out, bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) {
        cudaGetLastError();
        return HAG_ERR_CUDA;
    }
    return HAG_OK;
}

extern "C" int32_t hag_last_launch_count(const hag_t *h) { return h ? h->last_launches : 0; }

// ---- device-side check of the uploaded structure (a diagnostic: no gather kernel is involved) ----------------------
namespace {
__global__ void check_ids_kernel(const int32_t *ids, int64_t count, int32_t lo, int32_t hi, unsigned int bit, unsigned int *err) {
    for (int64_t i = blockIdx.x * int64_t(blockDim.x) + threadIdx.x; i < count; i += int64_t(gridDim.x) * blockDim.x)
        if (!hag_id_in_range(ids[i], lo, hi)) {
            atomicOr(err, bit);
            return;
        }
}
__global__ void check_ptr_kernel(const int32_t *ptr, int64_t rows, int32_t first, int32_t last, unsigned int bit, unsigned int *err) {
    for (int64_t i = blockIdx.x * int64_t(blockDim.x) + threadIdx.x; i <= rows; i += int64_t(gridDim.x) * blockDim.x)
        if (!hag_ptr_ok(i, rows, i ? ptr[i - 1] : 0, ptr[i], first, last)) {
            atomicOr(err, bit);
            return;
        }
}
}  // namespace

extern "C" hag_status hag_device_validate(hag_t *h, uint32_t *failed_lists, void *cuda_stream) {
    if (!h) return HAG_ERR_NULL;
    if (failed_lists) *failed_lists = 0;
    if (h->device < 0) return HAG_ERR_NOT_ON_DEVICE;
    hagl::DeviceGuard scope(h->device);
    if (!scope.ok) { cudaGetLastError(); return HAG_ERR_CUDA; }
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    unsigned int *err = nullptr;
    if (cudaMalloc(reinterpret_cast<void **>(&err), sizeof(unsigned int)) != cudaSuccess) { cudaGetLastError(); return HAG_ERR_OOM_DEVICE; }
    bool ok = cudaMemsetAsync(err, 0, sizeof(unsigned int), s) == cudaSuccess;
    const hag_device_arrays &d = h->d;
    const int32_t n = h->n, k = h->num_agg;
    auto grid_for = [](int64_t count) { return unsigned(std::max<int64_t>(1, std::min<int64_t>((count + 255) / 256, 1184))); };
    auto ids = [&](const int32_t *p, int64_t count, int32_t lo, int32_t hi, int list) {
        if (!ok || count <= 0 || !p) return;
        check_ids_kernel<<<grid_for(count), 256, 0, s>>>(p, count, lo, hi, 1u << list, err);
        ok = cudaGetLastError() == cudaSuccess;
    };
    auto ptrs = [&](const int32_t *p, int64_t rows, int64_t last, int list) {
        if (!ok || !p) return;
        check_ptr_kernel<<<grid_for(rows + 1), 256, 0, s>>>(p, rows, 0, int32_t(last), 1u << list, err);
        ok = cudaGetLastError() == cudaSuccess;
    };
    const int64_t f_rows = int64_t(h->ftail_ptr.size()) - 1, b_rows = int64_t(h->btail_ptr.size()) - 1;
    ids(d.agg_in, 2 * int64_t(k), 0, n + k, 0);
    ptrs(d.res_ptr, n, h->e_res, 1);
    ids(d.res_idx, h->e_res, 0, n + k, 1);
    ptrs(d.t_ptr, int64_t(n) + k, h->e_hat, 2);
    ids(d.t_idx, h->e_hat, 0, n + k, 2);
    ptrs(d.csr_ptr, n, h->e, 3);
    ids(d.csr_idx, h->e, 0, n, 3);
    ptrs(d.csr_t_ptr, n, h->e, 4);
    ids(d.csr_t_idx, h->e, 0, n, 4);
    if (f_rows > 0) {       // sources of an expanded node: the layer input and the levels up to the forward cut
        ptrs(d.ftail_ptr, f_rows, int64_t(h->ftail_idx.size()), 5);
        ids(d.ftail_idx, int64_t(h->ftail_idx.size()), 0, n + int32_t(h->level_ptr[h->fwd_cut]), 5);
    }
    if (b_rows > 0) {       // destinations of an expanded node: graph nodes only
        ptrs(d.btail_ptr, b_rows, int64_t(h->btail_idx.size()), 6);
        ids(d.btail_idx, int64_t(h->btail_idx.size()), 0, n, 6);
    }
    for (const seg_set *set : {&h->seg_res, &h->seg_t, &h->seg_csr, &h->seg_csr_t, &h->seg_ftail, &h->seg_btail})
        ids(set->d_order, int64_t(set->order.size()), set->order_first_row, set->order_first_row + int32_t(set->order.size()), 7);
    unsigned int host = 0;
    ok = ok && cudaMemcpyAsync(&host, err, sizeof(unsigned int), cudaMemcpyDeviceToHost, s) == cudaSuccess &&
         cudaStreamSynchronize(s) == cudaSuccess;
    cudaFree(err);
    if (!ok) { cudaGetLastError(); return HAG_ERR_CUDA; }
    if (failed_lists) *failed_lists = host;
    return host ? HAG_ERR_GRAPH : HAG_OK;
}

extern "C" hag_status hag_set_schedule(hag_t *h, int32_t schedule) {
    if (!h) return HAG_ERR_NULL;
    if (schedule < 0 || schedule > 2) return HAG_ERR_ARG;
    h->schedule = schedule;
    return HAG_OK;
}

extern "C" hag_status hag_device_status(hag_t *h) {
    if (!h) return HAG_ERR_NULL;
    if (h->device < 0 || !h->d.err_host) return HAG_ERR_NOT_ON_DEVICE;
    volatile unsigned int *w = h->d.err_host;
    if (*w == 0) return HAG_OK;
    *w = 0;
    return HAG_ERR_TIMEOUT;
}

// A one-CTA launch of the single-launch kernel over a two-phase list whose first phase is never
// finished by anybody: the one row item must run out of polls, record it, and still end.
extern "C" hag_status hag_selftest_wait_limit(hag_t *h, void *cuda_stream) {
    if (!h) return HAG_ERR_NULL;
    if (h->device < 0) return HAG_ERR_NOT_ON_DEVICE;
    DeviceGuard guard(h->device);
    if (!guard.ok) { cudaGetLastError(); return HAG_ERR_CUDA; }
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    constexpr int D = 4;
    struct Blob {
        int32_t items[16];
        int32_t phase_size[4];
        int32_t idx[4];
        unsigned int ctl[kFusedCtlWords];
        float prim[D], sec[D], out[D];
    } host{};
    const int32_t row_item[4] = {0, 1, 0, (0 + 1) | (1 << 8) | (1 << 16)};     // a row of phase 1 whose one entry is read after a wait for phase 0
    const int32_t pad_item[4] = {0, 0, -1, 0 | (1 << 8)};
    for (int i = 0; i < 4; ++i) {
        host.items[i] = row_item[i];
        for (int q = 1; q < 4; ++q) host.items[4 * q + i] = pad_item[i];
    }
    host.phase_size[0] = 4;      // four rows that nobody holds
    host.phase_size[1] = 4;
    host.idx[0] = 1;             // an aggregation-node id (n_prim = 1): the row must wait before it loads it
    Blob *dev = nullptr;
    if (cudaMalloc(reinterpret_cast<void **>(&dev), sizeof(Blob)) != cudaSuccess) { cudaGetLastError(); return HAG_ERR_OOM_DEVICE; }
    hag_status st = HAG_OK;
    if (cudaMemcpyAsync(dev, &host, sizeof(Blob), cudaMemcpyHostToDevice, s) != cudaSuccess) st = HAG_ERR_CUDA;
    if (st == HAG_OK) {
        hagk::FusedArgs k{};
        k.a.idx = dev->idx;
        k.a.prim = dev->prim;
        k.a.sec = dev->sec;
        k.a.n_prim = 1;
        k.a.out = dev->out;
        k.a.D = D;
        k.items = reinterpret_cast<const int4 *>(dev->items);
        k.n_items = 4;
        k.last_phase = 1;
        k.phase_size = dev->phase_size;
        k.ctl = dev->ctl;
        k.ahat = dev->sec;
        k.err_host = h->d.err_dev;
        k.spin_limit = 2000;     // a few milliseconds
        if (launch_pdl(hagk::fused_pass_kernel<float, 4, 4, false, 8, false>, 1u, k, s) != cudaSuccess) st = HAG_ERR_CUDA;
    }
    if (cudaStreamSynchronize(s) != cudaSuccess) st = HAG_ERR_CUDA;
    cudaFree(dev);
    if (st != HAG_OK) { cudaGetLastError(); return st; }
    return hag_device_status(h);
}

extern "C" hag_status hag_profile_enable(hag_t *h, int enable) {
    if (!h) return HAG_ERR_NULL;
    h->profile = enable != 0;
    return HAG_OK;
}

extern "C" int32_t hag_profile_read(hag_t *h, int32_t max, float *ms, int32_t *kind, int64_t *rows, int64_t *edges) {
    if (!h || h->device < 0) return -1;
    const int32_t count = int32_t(h->notes.size());
    if (!h->profile) return count;
    DeviceGuard guard(h->device);
    if (!guard.ok) { cudaGetLastError(); return -1; }
    for (int32_t i = 0; i < count && i < max; ++i) {
        if (h->events.size() < size_t(2 * (i + 1))) return -1;
        if (cudaEventSynchronize(h->events[2 * i + 1]) != cudaSuccess) { cudaGetLastError(); return -1; }
        float t = 0.f;
        if (cudaEventElapsedTime(&t, h->events[2 * i], h->events[2 * i + 1]) != cudaSuccess) { cudaGetLastError(); return -1; }
        if (ms) ms[i] = t;
        if (kind) kind[i] = h->notes[i].kind;
        if (rows) rows[i] = h->notes[i].rows;
        if (edges) edges[i] = h->notes[i].edges;
    }
    return count;
}

// --------------------------------------------------------------------------- //
// Forward pass without any allocation: the aggregation-node rows live in an
// array inside the library image.  Kept apart from the code above on purpose:
// it shares only the launch helpers.
// --------------------------------------------------------------------------- //
namespace {

// Device memory reserved on every GPU that loads this library, until exit.
static __device__ __align__(256) unsigned char g_static_scratch[HAG_STATIC_SCRATCH_BYTES];

constexpr int kMaxStaticDevices = 64;
// Device address of g_static_scratch per device ordinal.  In host code the name
// g_static_scratch is only a handle for the runtime, never an address a kernel
// may be given; the address comes from cudaGetSymbolAddress, once per device.
void *g_static_scratch_addr[kMaxStaticDevices] = {};

// Caller has made `device` current.
hag_status static_scratch_address(int device, void **out) {
    if (device < 0 || device >= kMaxStaticDevices) return HAG_ERR_ARG;
    void *p = __atomic_load_n(&g_static_scratch_addr[device], __ATOMIC_ACQUIRE);
    if (!p) {
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return HAG_ERR_CUDA;
        }
        __atomic_store_n(&g_static_scratch_addr[device], p, __ATOMIC_RELEASE);  // same value from any thread
    }
    *out = p;
    return HAG_OK;
}

// The same launch sequence as hag_aggregate_fwd, with no bookkeeping on the handle.
template <typename T>
hag_status fwd_static_impl(const hag *h, hag_reduce reduce, int32_t D, const void *x, void *out, float *scratch,
                           cudaStream_t s) {
    return fwd_impl<T>(h, true, reduce, D, x, out, scratch, s, nullptr);
}

}  // namespace

extern "C" hag_status hag_aggregate_fwd_static(const hag_t *h, hag_reduce reduce, hag_dtype dtype, int32_t D,
                                               const void *x, void *out, void *cuda_stream) {
    hag_status st = check_call(h, dtype, D, x, out);
    if (st != HAG_OK) return st;
    if (reduce != HAG_SUM && reduce != HAG_MEAN && reduce != HAG_GCN) return HAG_ERR_ARG;
    if (hag_workspace_bytes(h, D) > size_t(HAG_STATIC_SCRATCH_BYTES)) return HAG_ERR_TOO_LARGE;
    DeviceGuard guard(h->device);
    if (!guard.ok) { cudaGetLastError(); return HAG_ERR_CUDA; }
    void *scratch = nullptr;
    st = static_scratch_address(h->device, &scratch);
    if (st != HAG_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (dtype == HAG_F32) return fwd_static_impl<float>(h, reduce, D, x, out, static_cast<float *>(scratch), s);
    return fwd_static_impl<__nv_bfloat16>(h, reduce, D, x, out, static_cast<float *>(scratch), s);
}
