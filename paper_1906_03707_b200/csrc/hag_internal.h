// Internal definition of the opaque handle.  Host arrays are the canonical
// layout documented in include/hag.h; device arrays are their int32 copies.
#pragma once
#include <cstdint>
#include <vector>

#include <cuda_runtime.h>

#include "hag.h"

constexpr int kSchedSlots = 64;      // far more than the kernels that can overlap on one stream

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
    float *inv_degree = nullptr;   // [n] 1/|N(v)| (1 for empty rows)
    unsigned int *sched = nullptr; // ring of kSchedSlots (next row, finished warps) pairs, zero between launches
    // staging for the host-buffer entry point
    void *stage_in = nullptr;
    void *stage_out = nullptr;
    void *stage_ws = nullptr;
    size_t stage_in_bytes = 0, stage_out_bytes = 0, stage_ws_bytes = 0;
};

struct hag {
    int32_t n = 0, capacity = 0, num_agg = 0, num_levels = 0;
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

// hag_build.cpp: the search (Algorithm 3) in creation-id space.  Fills
// h->trace and returns the residual rows (creation ids, ascending) in
// rows_store/rows_len laid over the input row_ptr.
hag_status hag_search(hag *h, std::vector<int32_t> &rows_store, std::vector<int32_t> &rows_len);
// hag_build.cpp: levels, level-sorted renumbering, residual CSR, transposes, counters.
hag_status hag_layout(hag *h, const std::vector<int32_t> &rows_store, const std::vector<int32_t> &rows_len);
