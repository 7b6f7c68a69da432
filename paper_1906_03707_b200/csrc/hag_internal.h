// Internal definition of the opaque handle.  Host arrays are the canonical
// layout documented in include/hag.h; device arrays are their int32 copies.
#pragma once
#include <cstdint>
#include <vector>

#include <cuda_runtime.h>

#include "hag.h"

// Predicates of the device-side structure check (hag_device_validate), shared by its kernels and by the host test hook.
#if defined(__CUDACC__)
#define HAG_HOST_DEVICE __host__ __device__
#else
#define HAG_HOST_DEVICE
#endif
HAG_HOST_DEVICE inline bool hag_id_in_range(int32_t id, int32_t lo, int32_t hi) { return id >= lo && id < hi; }
// pointer i of a CSR-like list: the first is `first`, none steps back, the last is `last`
HAG_HOST_DEVICE inline bool hag_ptr_ok(int64_t i, int64_t rows, int32_t prev, int32_t cur, int32_t first, int32_t last) {
    return (i == 0 ? cur == first : cur >= prev) && (i < rows || cur == last);
}

// Segments of the long rows of one CSR-like table (see hag_kernels.cuh): host copy and device copy.
struct seg_table {
    std::vector<int32_t> segs;    // 4 per segment: row id, first entry, end entry, slot
    std::vector<int32_t> slots;   // 2 per long row: first segment, number of segments
    int32_t *d_segs = nullptr;
    int32_t *d_slots = nullptr;
    unsigned int *d_done = nullptr;
    int64_t count() const { return int64_t(segs.size() / 4); }
};

// Three granularities of splitting, chosen per launch by its number of rows: a launch that cannot fill the
// machine with whole rows is split finely (more parallel work, at the price of a partial row and a completion
// count per segment); a launch with rows to spare only splits what would otherwise stick out as a tail.
constexpr int kSegGrans = 3;
constexpr int32_t kSegLongRow[kSegGrans] = {64, 256, 1024};   // rows with more entries are split ...
constexpr int32_t kSegLength[kSegGrans] = {32, 128, 512};     // ... into segments of this many entries
inline int seg_gran_for_rows(int64_t rows) { return rows < 8192 ? 0 : (rows < 65536 ? 1 : 2); }

// Rows of like length side by side, for the kernels that walk several rows per warp in lock step: within windows of
// kOrderWindow rows (so that rows that share neighbours stay close in time) the rows are sorted by length, longest
// first.  order[r - first_row] is the row that takes the place of row r; windows never cross a boundary between
// launches (graph nodes | level 1 | level 2 ...), so every launch's range of rows maps onto itself.  Empty where the
// rows as they are lose less than kOrderMinWaste of the lock-step rounds.
constexpr int32_t kOrderWindow = 2048;
constexpr double kOrderMinWaste = 1.08;
constexpr int64_t kOrderNearRows = 8192;     // launches of aggregation-node rows from this size on are put in the order of their first entry

struct seg_set {
    seg_table g[kSegGrans];
    std::vector<int32_t> order;
    int32_t order_first_row = 0;
    int32_t *d_order = nullptr;
    int64_t max_count() const {
        int64_t m = 0;
        for (const seg_table &t : g) m = m > t.count() ? m : t.count();
        return m;
    }
};

constexpr int kSchedSlots = 64;      // far more than the kernels that can overlap on one stream

// One whole pass (all aggregation-node levels, then the graph nodes) as ONE launch of resident warps.
// The pass is a list of rows in dependency order: the rows of phase 0, then phase 1, ...; a phase is one
// level of aggregation nodes (as rows of two entries where the level is evaluated pair by pair), or the
// expanded deep nodes, or the chunk rows of the long rows of the phase after it, or (last) the graph-node
// rows.  Warps take rows in list order from a counter; a row that reads rows written by an earlier phase
// waits, with an iteration limit, until that phase's finished-row count is complete.  Because rows are
// handed out in list order, whatever a row waits for is already in the hands of a running warp, so the
// wait cannot deadlock.
constexpr int kFusedItemsPerGrab = 4;     // a grab never straddles two phases (phases are padded to it)
constexpr int kFusedMaxPhases = 56;       // deeper hierarchies run level by level
constexpr int64_t kFusedRowsForFullGrabs = 320000;   // phases with fewer rows are handed out two rows, below a quarter of it one row, per grab
constexpr int kFusedCtlWords = 64;        // per launch: [0] next row, [1] finished warps, [2] error, [4 + p] finished rows of phase p
constexpr int kFusedCtlSlots = 16;        // ring: consecutive launches (overlapping under programmatic dependent launch) take turns
constexpr int kFusedSpinLimit = 1 << 20;  // polls of a waiting warp, a microsecond apart, before it gives up (about a second)

struct fused_table {
    bool ok = false;                 // false: no row list (too many phases, or no rows); the id list is built all the same
    std::vector<int32_t> items;      // 4 per row: b, e, row, (required phase + 1) | phase << 8.  The row sums the entries [b, e) of
                                     // `ids` into output row `row` (row < 0: padding; row >= n: an aggregation node or a chunk row)
    std::vector<int32_t> phase_size; // rows per phase, padding included
    std::vector<int32_t> ids;        // the pass's id list: pair inputs, expansion lists, row lists, chunk ids of the long rows
    int64_t head_items = 0;          // rows of the list before the graph-node rows (and the chunk rows of their long rows): the
                                     // aggregation nodes' part of the pass, which can be launched by itself
    int64_t off_head = 0;            // where the expansion lists (ftail / btail) start in ids
    int64_t off_tail = 0;            // where the row lists (residual rows / transposed HAG / input graph) start
    int64_t n_chunks = 0;            // chunk rows: fp32 partial rows needed behind the aggregation nodes' rows
    int32_t last_phase = 0;          // the graph-node rows: nothing waits for them
    int64_t n_items() const { return int64_t(items.size() / 4); }
    int32_t *d_items = nullptr, *d_phase_size = nullptr, *d_ids = nullptr;
};

struct hag_device_arrays {
    // HAG
    int32_t *agg_in = nullptr;     // [2*num_agg]
    int32_t *res_ptr = nullptr;    // [n+1]
    int32_t *res_idx = nullptr;    // [e_res]
    int32_t *t_ptr = nullptr;      // [n+num_agg+1]
    int32_t *t_idx = nullptr;      // [e_hat]
    // input graph and its transpose
    int32_t *csr_ptr = nullptr;    // [n+1]
    int32_t *csr_idx = nullptr;    // [e]
    int32_t *csr_t_ptr = nullptr;  // [n+1]
    int32_t *csr_t_idx = nullptr;  // [e]
    int32_t *ftail_ptr = nullptr, *ftail_idx = nullptr;   // forward expansion of the deep levels
    int32_t *btail_ptr = nullptr, *btail_idx = nullptr;   // backward expansion
    // res_idx, t_idx, csr_idx, csr_t_idx and the expansion lists above point into the id lists of the four passes
    // (fused_table::d_ids), which hold them next to what else a single-launch pass reads
    unsigned int *fused_ctl = nullptr;     // kFusedCtlSlots x kFusedCtlWords, zero between launches
    unsigned int *err_host = nullptr;      // one word of mapped pinned host memory: set by a kernel whose wait ran out
    unsigned int *err_dev = nullptr;       // its device address
    float *inv_degree = nullptr;   // [n] 1/|N(v)| (1 for empty rows)
    float *inv_degree1 = nullptr;  // [n] 1/(|N(v)| + 1): the GCN normalisation
    unsigned int *sched = nullptr; // ring of kSchedSlots (next row, finished warps) pairs, zero between launches
    // staging for the host-buffer entry point: the input side is double-buffered and copied on a stream of its
    // own, so that the copy-in of one call runs under the aggregation and the copy-out of the call before it
    void *stage_in = nullptr;
    void *stage_in2 = nullptr;
    void *stage_out = nullptr;
    void *stage_ws = nullptr;
    size_t stage_in_bytes = 0, stage_in2_bytes = 0, stage_out_bytes = 0, stage_ws_bytes = 0;
    cudaStream_t copy_in_stream = nullptr;
    cudaEvent_t in_ready[2] = {nullptr, nullptr};   // copy-in into buffer i finished
    cudaEvent_t in_free[2] = {nullptr, nullptr};    // the aggregation that read buffer i finished
    uint32_t host_calls = 0;
};

struct hag {
    int32_t n = 0, capacity = 0, num_agg = 0, num_levels = 0;
    int32_t min_redundancy = 2;      // the search stops below this redundancy (2 = the paper's "> 1")
    int64_t e = 0, e_res = 0, e_hat = 0;
    std::vector<int64_t> csr_ptr;
    std::vector<int32_t> csr_idx;
    std::vector<int64_t> csr_t_ptr;
    std::vector<int32_t> csr_t_idx;
    std::vector<int32_t> in_degree;
    std::vector<int32_t> trace;      // 3 * num_agg: v1, v2 (creation ids), redundancy
    std::vector<int64_t> level_ptr;  // num_levels + 1
    std::vector<int32_t> agg_in;     // 2 * num_agg
    std::vector<int64_t> res_ptr;    // n + 1
    std::vector<int32_t> res_idx;
    std::vector<int64_t> t_ptr;      // n + num_agg + 1
    std::vector<int32_t> t_idx;
    // deep levels expanded (one launch each way)
    int32_t fwd_cut = 0, bwd_cut = 0;
    std::vector<int64_t> ftail_ptr, btail_ptr;
    std::vector<int32_t> ftail_idx, btail_idx;
    seg_set seg_res, seg_t, seg_csr, seg_csr_t, seg_ftail, seg_btail;
    fused_table fz_fwd, fz_bwd, fz_csr, fz_csr_t;   // the four passes as single launches
    int32_t schedule = 0;            // 0: a launch per level; 1: one launch per pass where a row list exists
    uint32_t fused_seq = 0;          // next slot of the control ring
    int32_t spin_limit = kFusedSpinLimit;
    int64_t max_segs_hag = 0, max_segs_csr = 0;   // partial rows the HAG / plain calls need in the workspace
    hag_info info{};
    int device = -1;
    hag_device_arrays d;
    int32_t last_launches = 0;
    int32_t sm_count = 0;            // of the device holding the arrays
    uint32_t sched_seq = 0;          // next slot of the scheduling ring
    // per-launch timing (hag_profile_*)
    bool profile = false;
    std::vector<cudaEvent_t> events;          // pairs: 2*i start, 2*i+1 stop
    struct launch_note { int32_t kind; int64_t rows, edges; };
    std::vector<launch_note> notes;           // launches of the last call
};

// Allocation-failure injection for tests (hag_test_fail_allocation): true when the allocation attempt that is
// about to be made is the one chosen to fail.  kind 0: host memory, 1: device memory.
bool hag_alloc_should_fail(int kind);

// hag_build.cpp: the search (Algorithm 3) in creation-id space.  Fills
// h->trace and returns the residual rows (creation ids, ascending) in
// rows_store/rows_len laid over the input row_ptr.
hag_status hag_search(hag *h, std::vector<int32_t> &rows_store, std::vector<int32_t> &rows_len);
// hag_build.cpp: levels, level-sorted renumbering, residual CSR, transposes, counters.
hag_status hag_layout(hag *h, const std::vector<int32_t> &rows_store, const std::vector<int32_t> &rows_len);
