// hag_build: the HAG search of Algorithm 3 (set Aggregate) and the device layout.
//
// The search is exact: every iteration merges the pair with the largest
// Redundancy (number of graph nodes aggregating both), ties to the smallest
// (v1, v2).  Instead of a count per pair (billions at the larger shapes) it
// keeps, per node x, key[x] >= max_b Redundancy(x, b) together with a partner
// and a "dirty" flag:
//   * a merge of (v1, v2) with users U changes only pairs that contain v1 or v2
//     (they lose |U n out(y)|) and creates pairs (y, w) with count |U n out(y)|,
//     which never exceeds the old count of (y, v1).  So no key ever has to rise,
//     a node whose recorded partner is neither v1 nor v2 keeps an exact key, and
//     the new node's key is known exactly from the same pass;
//   * nodes whose partner was merged away are only marked dirty; their key stays
//     a valid upper bound and is recounted when it reaches the top of the queue.
// The queue is ordered by (key descending, id ascending); a clean top is the
// arg-max with the required tie-break (its partner is the smallest id attaining
// the count, and is larger than the node itself, otherwise the partner would
// have been on top).  Memory is O(|E|).
// Recounts are nine tenths of the time and independent of each other while no
// merge happens, so a run of stale nodes at the top of the queue is recounted
// by a pool of threads at once.  Recounting a stale node early only tightens a
// bound sooner: the merge sequence is the same for any number of threads.
#include <algorithm>
#include <limits>
#include <atomic>
#include <chrono>
#include <cstring>
#include <new>
#include <queue>
#include <thread>

#include "hag_internal.h"

namespace {

std::atomic<int> g_build_threads{0};   // 0 = as many as the host has, at most 16

struct Searcher {
    int32_t n;
    int64_t cap;
    const int64_t *row_ptr;
    std::vector<int32_t> &rows;      // row u: rows[row_ptr[u] .. row_ptr[u] + row_len[u])
    std::vector<int32_t> &row_len;
    std::vector<int32_t> out_store;  // users of the graph nodes, grouped by source
    std::vector<int32_t *> out_ptr;  // per id
    std::vector<int32_t> out_len;
    std::vector<std::vector<int32_t>> out_new;  // storage for aggregation nodes' user lists
    std::vector<int32_t> key, partner;
    std::vector<uint8_t> dirty;
    std::vector<int32_t> cnt, touched, users;
    std::priority_queue<uint64_t> pq;

    Searcher(int32_t n_, int64_t cap_, const int64_t *rp, std::vector<int32_t> &r, std::vector<int32_t> &rl)
        : n(n_), cap(cap_), row_ptr(rp), rows(r), row_len(rl) {}

    static uint64_t enc(int32_t k, int32_t id) { return (uint64_t(uint32_t(k)) << 32) | uint32_t(0x7fffffff - id); }

    // exact max_b Redundancy(x, b) and the smallest b attaining it (reads shared state only)
    void recount(int32_t x, int32_t &best, int32_t &arg, std::vector<int32_t> &cnt, std::vector<int32_t> &touched) const {
        touched.clear();
        const int32_t *ou = out_ptr[x];
        for (int32_t i = 0, m = out_len[x]; i < m; ++i) {
            const int32_t u = ou[i];
            const int32_t *row = rows.data() + row_ptr[u];
            for (int32_t j = 0, l = row_len[u]; j < l; ++j) {
                const int32_t y = row[j];
                if (cnt[y]++ == 0) touched.push_back(y);
            }
        }
        best = 0;
        arg = -1;
        for (int32_t y : touched) {
            const int32_t c = cnt[y];
            cnt[y] = 0;
            if (y == x) continue;
            if (c > best || (c == best && y < arg)) { best = c; arg = y; }
        }
    }

    // Re-applies the first `count` merges of a recorded trace (no search).
    hag_status replay(const std::vector<int32_t> &src, int64_t count, std::vector<int32_t> &trace) {
        init_lists();
        for (int64_t i = 0; i < count; ++i) {
            const int32_t x = src[3 * i], p = src[3 * i + 1], k = src[3 * i + 2];
            if (!(0 <= x && x < p && p < n + i)) return HAG_ERR_ARG;
            intersect_users(x, p);
            if (int32_t(users.size()) != k) return HAG_ERR_ARG;
            int32_t wbest, warg;
            apply_merge(x, p, i, trace, wbest, warg);
        }
        return HAG_OK;
    }

    void init_lists() {
        const int64_t n_ids = int64_t(n) + cap;
        const int64_t e = row_ptr[n];
        out_ptr.assign(n_ids, nullptr);
        out_len.assign(n_ids, 0);
        key.assign(n_ids, 0);
        partner.assign(n_ids, -1);
        dirty.assign(n_ids, 0);
        cnt.assign(n_ids, 0);
        out_new.resize(cap);
        out_store.resize(e > 0 ? e : 1);
        users.reserve(1024);
        {   // users of every graph node as a source: transpose of the rows
            std::vector<int64_t> off(n + 1, 0);
            for (int64_t i = 0; i < e; ++i) off[rows[i] + 1]++;
            for (int32_t s = 0; s < n; ++s) off[s + 1] += off[s];
            for (int32_t s = 0; s < n; ++s) out_ptr[s] = out_store.data() + off[s];
            for (int32_t u = 0; u < n; ++u)
                for (int64_t i = row_ptr[u]; i < row_ptr[u + 1]; ++i) {
                    const int32_t s = rows[i];
                    out_ptr[s][out_len[s]++] = u;
                }
        }
    }

    // users <- the graph nodes that hold both x and p
    void intersect_users(int32_t x, int32_t p) {
        users.clear();
        const int32_t *a = out_ptr[x], *b = out_ptr[p];
        int32_t i = 0, j = 0;
        const int32_t la = out_len[x], lb = out_len[p];
        while (i < la && j < lb) {
            if (a[i] < b[j]) ++i;
            else if (a[i] > b[j]) ++j;
            else { users.push_back(a[i]); ++i; ++j; }
        }
    }

    // Merge (x, p) with the users already in `users` into node n + num: rewrites the
    // rows and user lists, marks what became stale, returns the new node's exact key.
    void apply_merge(int32_t x, int32_t p, int64_t num, std::vector<int32_t> &trace, int32_t &wbest, int32_t &warg) {
        const int32_t w = int32_t(n + num);
        trace.push_back(x);
        trace.push_back(p);
        trace.push_back(int32_t(users.size()));
        // rewrite the users' rows; count what else they hold (= the new node's pair counts)
        touched.clear();
        for (int32_t u : users) {
            int32_t *row = rows.data() + row_ptr[u];
            const int32_t l = row_len[u];
            int32_t o = 0;
            for (int32_t j = 0; j < l; ++j) {
                const int32_t y = row[j];
                if (y == x || y == p) continue;
                row[o++] = y;
                if (cnt[y]++ == 0) touched.push_back(y);
            }
            row[o++] = w;                       // larger than every existing id: row stays sorted
            row_len[u] = o;
        }
        wbest = 0;
        warg = -1;
        for (int32_t y : touched) {
            const int32_t c = cnt[y];
            cnt[y] = 0;
            if (c > wbest || (c == wbest && y < warg)) { wbest = c; warg = y; }
            if (!dirty[y] && (partner[y] == x || partner[y] == p)) dirty[y] = 1;
        }
        // user lists: x and p lose U, w gets it
        for (int32_t s : {x, p}) {
            int32_t *l = out_ptr[s];
            const int32_t len = out_len[s];
            int32_t o = 0;
            size_t q = 0;
            for (int32_t i = 0; i < len; ++i) {
                while (q < users.size() && users[q] < l[i]) ++q;
                if (q < users.size() && users[q] == l[i]) continue;
                l[o++] = l[i];
            }
            out_len[s] = o;
        }
        out_new[num] = users;
        out_ptr[w] = out_new[num].data();
        out_len[w] = int32_t(users.size());
    }

    // ---- pool for batches of recounts ----
    int n_threads = 1;
    std::vector<std::thread> workers;
    std::vector<std::vector<int32_t>> w_cnt, w_touched;   // scratch per worker (index 0 = calling thread)
    std::vector<int32_t> batch, batch_best, batch_arg;
    std::atomic<int64_t> generation{0};
    std::atomic<int32_t> next_task{0}, tasks_done{0}, acks{0};
    std::atomic<bool> stop{false};

    void work_on_batch(int self) {
        const int32_t total = int32_t(batch.size());
        for (;;) {
            const int32_t i = next_task.fetch_add(1, std::memory_order_relaxed);
            if (i >= total) break;
            recount(batch[i], batch_best[i], batch_arg[i], w_cnt[self], w_touched[self]);
            tasks_done.fetch_add(1, std::memory_order_release);
        }
    }
    void worker_loop(int self) {
        int64_t seen = 0;
        for (;;) {
            int spins = 0;
            while (generation.load(std::memory_order_acquire) == seen) {
                if (stop.load(std::memory_order_acquire)) return;
                if (++spins > 2000) std::this_thread::yield();
            }
            seen = generation.load(std::memory_order_acquire);
            work_on_batch(self);
            acks.fetch_add(1, std::memory_order_release);   // this worker no longer touches the batch
        }
    }
    void start_pool(int threads) {
        n_threads = std::max(1, threads);
        w_cnt.assign(n_threads, std::vector<int32_t>());
        w_touched.assign(n_threads, std::vector<int32_t>());
        for (int t = 0; t < n_threads; ++t) w_cnt[t].assign(size_t(n) + cap, 0);
        for (int t = 1; t < n_threads; ++t) workers.emplace_back([this, t] { worker_loop(t); });
    }
    void stop_pool() {
        stop.store(true, std::memory_order_release);
        for (auto &t : workers) t.join();
        workers.clear();
    }
    // recounts every node of `batch` (all threads), results in batch_best / batch_arg
    void recount_batch() {
        const int32_t total = int32_t(batch.size());
        batch_best.assign(total, 0);
        batch_arg.assign(total, -1);
        next_task.store(0, std::memory_order_relaxed);
        tasks_done.store(0, std::memory_order_relaxed);
        const bool shared = n_threads > 1 && total > 1;
        if (shared) {
            acks.store(0, std::memory_order_relaxed);
            generation.fetch_add(1, std::memory_order_release);
        }
        work_on_batch(0);
        while (tasks_done.load(std::memory_order_acquire) < total) std::this_thread::yield();
        // the batch vectors are rebuilt next: wait until every worker has left this one
        if (shared)
            while (acks.load(std::memory_order_acquire) < n_threads - 1) std::this_thread::yield();
    }
    ~Searcher() { stop_pool(); }

    hag_status run(std::vector<int32_t> &trace, int threads, int32_t min_redundancy) {
        init_lists();
        start_pool(threads);
        const size_t max_batch = size_t(4) * n_threads;
        // a pair cannot be shared by more rows than either member has users
        for (int32_t s = 0; s < n; ++s) {
            key[s] = out_len[s];
            dirty[s] = 1;
            if (key[s] >= 2) pq.push(enc(key[s], s));
        }
        int64_t num = 0;
        while (num < cap && !pq.empty()) {
            const uint64_t top = pq.top();
            pq.pop();
            const int32_t k = int32_t(top >> 32);
            const int32_t x = int32_t(0x7fffffff - uint32_t(top & 0xffffffffu));
            if (k != key[x]) continue;              // superseded entry
            if (k < min_redundancy) break;           // every bound is below the stop value: so is every pair
            if (dirty[x]) {
                // gather the run of stale nodes at the top of the queue and recount them together
                batch.clear();
                batch.push_back(x);
                while (batch.size() < max_batch && !pq.empty()) {
                    const uint64_t t2 = pq.top();
                    const int32_t k2 = int32_t(t2 >> 32);
                    const int32_t x2 = int32_t(0x7fffffff - uint32_t(t2 & 0xffffffffu));
                    if (k2 != key[x2]) { pq.pop(); continue; }      // superseded entry
                    if (!dirty[x2] || k2 < 2) break;                // a clean node: stop before it
                    pq.pop();
                    dirty[x2] = 2;                                  // in the batch (guards against duplicate entries)
                    batch.push_back(x2);
                }
                dirty[x] = 2;
                // drop duplicates of one node (several live entries with the same key)
                std::sort(batch.begin(), batch.end());
                batch.erase(std::unique(batch.begin(), batch.end()), batch.end());
                recount_batch();
                for (size_t i = 0; i < batch.size(); ++i) {
                    const int32_t y = batch[i];
                    key[y] = batch_best[i];
                    partner[y] = batch_arg[i];
                    dirty[y] = 0;
                    if (key[y] >= 2) pq.push(enc(key[y], y));
                }
                continue;
            }
            const int32_t p = partner[x];
            if (p <= x) return HAG_ERR_ARG;         // cannot happen (see header comment)
            intersect_users(x, p);
            if (int32_t(users.size()) != k) return HAG_ERR_ARG;  // internal inconsistency
            int32_t wbest, warg;
            apply_merge(x, p, num, trace, wbest, warg);
            const int32_t w = int32_t(n + num);
            for (int32_t s : {x, p}) {
                dirty[s] = 1;                        // every pair with x or p changed
                const int32_t bound = std::min(key[s], out_len[s]);
                // x's entry was popped; p still has one unless its bound moved
                if ((s == x || bound != key[s]) && bound >= 2) pq.push(enc(bound, s));
                key[s] = bound;
            }
            key[w] = wbest;
            partner[w] = warg;
            dirty[w] = 0;
            if (wbest >= 2) pq.push(enc(wbest, w));
            ++num;
        }
        return HAG_OK;
    }
};

}  // namespace

namespace {
std::atomic<int> g_fail_countdown[2] = {{-1}, {-1}};
}

bool hag_alloc_should_fail(int kind) {
    int v = g_fail_countdown[kind].load();
    while (v >= 0)
        if (g_fail_countdown[kind].compare_exchange_weak(v, v - 1)) return v == 0;
    return false;
}

extern "C" hag_status hag_test_fail_allocation(int32_t kind, int32_t countdown) {
    if (kind != 0 && kind != 1) return HAG_ERR_ARG;
    g_fail_countdown[kind].store(countdown < 0 ? -1 : countdown);
    return HAG_OK;
}

hag_status hag_search(hag *h, std::vector<int32_t> &rows_store, std::vector<int32_t> &rows_len) {
    try {
        if (hag_alloc_should_fail(0)) throw std::bad_alloc();
        rows_store = h->csr_idx;
        rows_len.resize(h->n);
        for (int32_t u = 0; u < h->n; ++u) rows_len[u] = int32_t(h->csr_ptr[u + 1] - h->csr_ptr[u]);
        h->trace.clear();
        if (h->capacity == 0 || h->n == 0) return HAG_OK;
        Searcher s(h->n, h->capacity, h->csr_ptr.data(), rows_store, rows_len);
        int threads = g_build_threads.load();
        if (threads <= 0) threads = int(std::min<unsigned>(std::max<unsigned>(std::thread::hardware_concurrency(), 1u), 16u));
        hag_status st = s.run(h->trace, threads, h->min_redundancy);
        if (st != HAG_OK) return st;
    } catch (const std::bad_alloc &) {
        return HAG_ERR_OOM_HOST;
    }
    h->num_agg = int32_t(h->trace.size() / 3);
    return HAG_OK;
}

namespace {

// Deep levels without their intermediate nodes (Section 3.1, Eq. 1: aggr(v) aggregates cover(v)).
// Forward, cut c: every node deeper than level c gets the list of its cover restricted to ids of
// level <= c.  Backward, cut c: every node deeper than c gets the graph-node outputs that use it,
// directly or through deeper nodes.  Any 0 <= c <= L gives the same values; which one is taken is
// a question of launch cost only (choose_cuts).
void expand_tails(hag *h, int32_t fwd_cut, int32_t bwd_cut) {
    const int32_t n = h->n, k = h->num_agg, L = h->num_levels;
    std::vector<int32_t> clevel(k);      // level per canonical aggregation node
    for (int32_t l = 1; l <= L; ++l)
        for (int64_t j = h->level_ptr[l - 1]; j < h->level_ptr[l]; ++j) clevel[j] = l;
    auto level_of = [&](int32_t id) { return id < n ? 0 : clevel[id - n]; };
    h->fwd_cut = fwd_cut;
    {
        const int64_t j0 = h->level_ptr[fwd_cut];
        std::vector<std::vector<int32_t>> lists(size_t(k - j0));
        h->ftail_ptr.assign(size_t(k - j0) + 1, 0);
        for (int64_t j = j0; j < k; ++j) {
            std::vector<int32_t> &dst = lists[j - j0];
            for (int q = 0; q < 2; ++q) {
                const int32_t in = h->agg_in[2 * j + q];
                if (level_of(in) <= fwd_cut) dst.push_back(in);
                else dst.insert(dst.end(), lists[in - n - j0].begin(), lists[in - n - j0].end());
            }
            std::sort(dst.begin(), dst.end());
            h->ftail_ptr[j - j0 + 1] = h->ftail_ptr[j - j0] + int64_t(dst.size());
        }
        h->ftail_idx.clear();
        h->ftail_idx.reserve(size_t(h->ftail_ptr.back()));
        for (auto &l : lists) h->ftail_idx.insert(h->ftail_idx.end(), l.begin(), l.end());
    }
    h->bwd_cut = bwd_cut;
    {
        const int64_t j0 = h->level_ptr[bwd_cut];
        std::vector<std::vector<int32_t>> lists(size_t(k - j0));
        for (int64_t j = k - 1; j >= j0; --j) {
            std::vector<int32_t> &dst = lists[j - j0];
            for (int64_t i = h->t_ptr[n + j]; i < h->t_ptr[n + j + 1]; ++i) {
                const int32_t d = h->t_idx[i];
                if (d < n) dst.push_back(d);
                else dst.insert(dst.end(), lists[d - n - j0].begin(), lists[d - n - j0].end());
            }
            std::sort(dst.begin(), dst.end());
        }
        h->btail_ptr.assign(size_t(k - j0) + 1, 0);
        for (int64_t j = j0; j < k; ++j) h->btail_ptr[j - j0 + 1] = h->btail_ptr[j - j0] + int64_t(lists[j - j0].size());
        h->btail_idx.clear();
        h->btail_idx.reserve(size_t(h->btail_ptr.back()));
        for (auto &l : lists) h->btail_idx.insert(h->btail_idx.end(), l.begin(), l.end());
    }
}

// The cuts by launch cost.  What one extra launch costs, in rows moved; measured on B200: the
// backward launches (rows of tens of users each) pay for a merge up to four times later than the
// forward ones (rows of two to eight inputs).
void choose_cuts(const hag *h, int32_t &fwd_cut, int32_t &bwd_cut) {
    const int64_t kLaunchRows = 32768, kBwdLaunchRows = 131072;
    const int32_t n = h->n, k = h->num_agg, L = h->num_levels;
    std::vector<int32_t> clevel(k);
    for (int32_t l = 1; l <= L; ++l)
        for (int64_t j = h->level_ptr[l - 1]; j < h->level_ptr[l]; ++j) clevel[j] = l;
    auto level_of = [&](int32_t id) { return id < n ? 0 : clevel[id - n]; };
    // forward: size of the expansion of every node for a given cut
    int32_t best_c = L;
    int64_t best_cost = kLaunchRows * L;
    std::vector<int64_t> sz(k);
    for (int32_t c = L - 1; c >= 0; --c) {
        int64_t extra = 0;
        for (int64_t j = h->level_ptr[c]; j < k; ++j) {
            int64_t t = 0;
            for (int q = 0; q < 2; ++q) {
                const int32_t in = h->agg_in[2 * j + q];
                t += level_of(in) <= c ? 1 : sz[in - n];
            }
            sz[j] = t;
            extra += t - 1;
        }
        const int64_t cost = kLaunchRows * (c + 1) + extra;
        if (cost < best_cost) { best_cost = cost; best_c = c; }
    }
    fwd_cut = best_c;
    // backward: every node's transitive graph-node users (independent of the cut)
    std::vector<int64_t> usz(k);
    for (int64_t j = k - 1; j >= 0; --j) {
        int64_t t = 0;
        for (int64_t i = h->t_ptr[n + j]; i < h->t_ptr[n + j + 1]; ++i) {
            const int32_t d = h->t_idx[i];
            t += d < n ? 1 : usz[d - n];
        }
        usz[j] = t;
    }
    int32_t best_b = L;
    int64_t best_bcost = kBwdLaunchRows * L;
    int64_t extra = 0;
    for (int32_t c = L - 1; c >= 0; --c) {
        for (int64_t j = h->level_ptr[c]; j < h->level_ptr[c + 1]; ++j)
            extra += usz[j] - (h->t_ptr[n + j + 1] - h->t_ptr[n + j]);
        const int64_t cost = kBwdLaunchRows * (c + 1) + extra;
        if (cost < best_bcost) { best_bcost = cost; best_b = c; }
    }
    bwd_cut = best_b;
}

// Segments of the long rows of every table the gather walks.
void build_segments(hag *h) {
    const int32_t n = h->n, k = h->num_agg;
    auto build = [](seg_set &set, const std::vector<int64_t> &ptr, int64_t rows, int32_t first_row_id) {
        for (int gran = 0; gran < kSegGrans; ++gran) {
            seg_table &t = set.g[gran];
            const int64_t long_row = kSegLongRow[gran], seg_len = kSegLength[gran];
            t.segs.clear();
            t.slots.clear();
            for (int64_t r = 0; r < rows; ++r) {
                const int64_t b = ptr[r], e = ptr[r + 1];
                if (e - b <= long_row) continue;
                const int32_t slot = int32_t(t.slots.size() / 2);
                const int32_t first = int32_t(t.segs.size() / 4);
                int32_t n_seg = 0;
                for (int64_t sb = b; sb < e; sb += seg_len, ++n_seg) {
                    t.segs.push_back(int32_t(first_row_id + r));
                    t.segs.push_back(int32_t(sb));
                    t.segs.push_back(int32_t(std::min<int64_t>(sb + seg_len, e)));
                    t.segs.push_back(slot);
                }
                t.slots.push_back(first);
                t.slots.push_back(n_seg);
            }
        }
    };
    // the row order of the several-rows-per-warp kernels (see seg_set); `bounds`: ascending local row indices where
    // launches begin (0 and rows included)
    // `near_from`: from this segment of `bounds` on the rows are aggregation nodes, whose ids follow the order of the
    // search, not of the graph: those segments are first put in the order of their first entry (rows that read the same
    // neighbourhood side by side, so that what one row brings into the L2 the next ones find there), then sorted by
    // length within the windows.  Segments of fewer than kOrderNearRows rows stay as they are (their launches are bound
    // by latency, and the order costs a dependent load).
    auto order = [](seg_set &set, const std::vector<int64_t> &ptr, const std::vector<int32_t> &idx, int64_t rows, int32_t first_row_id,
                    const std::vector<int64_t> &bounds, size_t near_from) {
        set.order.clear();
        set.order_first_row = first_row_id;
        if (rows < 2) return;
        auto rounds = [&](int64_t r) { return (ptr[r + 1] - ptr[r] + 3) / 4; };
        int64_t own = 0, paired = 0;
        for (int64_t r = 0; r < rows; r += 2) {
            const int64_t a = rounds(r), b = r + 1 < rows ? rounds(r + 1) : 0;
            own += a + b;
            paired += 2 * std::max(a, b);
        }
        bool any_near = false;
        for (size_t i = near_from; i + 1 < bounds.size(); ++i) any_near = any_near || bounds[i + 1] - bounds[i] >= kOrderNearRows;
        const bool by_length = double(paired) >= kOrderMinWaste * double(std::max<int64_t>(own, 1));
        if (!by_length && !any_near) return;
        set.order.resize(size_t(rows));
        for (int64_t r = 0; r < rows; ++r) set.order[size_t(r)] = int32_t(first_row_id + r);
        auto len_of = [&](int32_t x) { return ptr[x - first_row_id + 1] - ptr[x - first_row_id]; };
        auto key_of = [&](int32_t x) {
            const int64_t r = x - first_row_id;
            return ptr[r] < ptr[r + 1] ? idx[size_t(ptr[r])] : std::numeric_limits<int32_t>::max();
        };
        for (size_t i = 0; i + 1 < bounds.size(); ++i) {
            const bool near = i >= near_from && bounds[i + 1] - bounds[i] >= kOrderNearRows;
            if (near)
                std::stable_sort(set.order.begin() + bounds[i], set.order.begin() + bounds[i + 1],
                                 [&](int32_t x, int32_t y) { return key_of(x) < key_of(y); });
            if (!by_length && !near) continue;
            for (int64_t w0 = bounds[i]; w0 < bounds[i + 1]; w0 += kOrderWindow) {
                const int64_t w1 = std::min<int64_t>(w0 + kOrderWindow, bounds[i + 1]);
                std::stable_sort(set.order.begin() + w0, set.order.begin() + w1, [&](int32_t x, int32_t y) { return len_of(x) > len_of(y); });
            }
        }
    };
    std::vector<int64_t> t_bounds{0, n};
    for (size_t l = 1; l < h->level_ptr.size(); ++l) t_bounds.push_back(n + h->level_ptr[l]);
    const int64_t f_rows = int64_t(h->ftail_ptr.size()) - 1, b_rows = int64_t(h->btail_ptr.size()) - 1;
    build(h->seg_res, h->res_ptr, n, 0);
    build(h->seg_t, h->t_ptr, int64_t(n) + k, 0);
    build(h->seg_csr, h->csr_ptr, n, 0);
    build(h->seg_csr_t, h->csr_t_ptr, n, 0);
    build(h->seg_ftail, h->ftail_ptr, f_rows, int32_t(n + h->level_ptr[h->fwd_cut]));
    build(h->seg_btail, h->btail_ptr, b_rows, int32_t(n + h->level_ptr[h->bwd_cut]));
    constexpr size_t kNone = size_t(1) << 30;
    order(h->seg_res, h->res_ptr, h->res_idx, n, 0, {0, n}, kNone);
    order(h->seg_t, h->t_ptr, h->t_idx, int64_t(n) + k, 0, t_bounds, 1);
    order(h->seg_csr, h->csr_ptr, h->csr_idx, n, 0, {0, n}, kNone);
    order(h->seg_csr_t, h->csr_t_ptr, h->csr_t_idx, n, 0, {0, n}, kNone);
    order(h->seg_ftail, h->ftail_ptr, h->ftail_idx, f_rows, int32_t(n + h->level_ptr[h->fwd_cut]), {0, std::max<int64_t>(f_rows, 0)}, 0);
    order(h->seg_btail, h->btail_ptr, h->btail_idx, b_rows, int32_t(n + h->level_ptr[h->bwd_cut]), {0, std::max<int64_t>(b_rows, 0)}, 0);
    h->max_segs_hag = std::max(std::max(h->seg_res.max_count(), h->seg_t.max_count()),
                               std::max(h->seg_ftail.max_count(), h->seg_btail.max_count()));
    h->max_segs_csr = std::max(h->seg_csr.max_count(), h->seg_csr_t.max_count());
}


// The four passes as row lists for the single-launch kernel (see hag_internal.h).
// How long a row may get before it is cut into chunk rows, by the size of the pass: a pass that cannot keep
// the machine busy for long must not end on one warp walking a hub row.
struct FusedSplit { int64_t long_row, chunk_len; };
FusedSplit fused_split_for_entries(int64_t entries) {
    if (entries < (int64_t(1) << 20)) return {64, 32};
    if (entries < (int64_t(16) << 20)) return {128, 64};
    return {1024, 512};
}

struct FusedBuilder {
    fused_table &t;
    const int32_t n, k;                 // graph nodes, aggregation nodes: chunk rows get the ids n + k, n + k + 1, ...
    const FusedSplit split;
    int32_t phase = -1;
    int64_t phase_begin = 0;
    FusedBuilder(fused_table &t_, int32_t n_, int32_t k_, FusedSplit sp) : t(t_), n(n_), k(k_), split(sp) { t = fused_table{}; }
    // n_sec: how many of the row's entries (its last ones) are rows that this launch writes: read after the wait
    void push(int64_t b, int64_t e, int32_t row, int req, int64_t n_sec = 0) {
        t.items.push_back(int32_t(b));
        t.items.push_back(int32_t(e));
        t.items.push_back(row);
        t.items.push_back(int32_t(uint32_t(req + 1) | (uint32_t(phase) << 8) | (uint32_t(req >= 0 ? n_sec : 0) << 16)));
    }
    // Rows per grab of four list slots, by the size of the phase: a phase that gives every resident warp only a
    // few grabs is handed out one row at a time (the other three slots are padding), or it would end on warps that
    // still have three rows to go while the rest wait for the phase to complete.
    int real_per_grab = kFusedItemsPerGrab, in_grab = 0;
    void begin_phase(int64_t rows = -1) {
        ++phase;
        phase_begin = t.n_items();
        in_grab = 0;
        real_per_grab = rows < 0 || rows >= kFusedRowsForFullGrabs ? 4 : (rows >= kFusedRowsForFullGrabs / 4 ? 2 : 1);
    }
    void push_row(int64_t b, int64_t e, int32_t row, int req, int64_t n_sec) {
        push(b, e, row, req, n_sec);
        if (++in_grab == real_per_grab) {
            while (t.n_items() % kFusedItemsPerGrab) push(0, 0, -1, -1);
            in_grab = 0;
        }
    }
    void end_phase() {
        while ((t.n_items() - phase_begin) % kFusedItemsPerGrab) push(0, 0, -1, -1);
        t.phase_size.push_back(int32_t(t.n_items() - phase_begin));
    }
    // Appends `ids` to the pass's id list and returns where they start.
    int64_t add_ids(const int32_t *ids, int64_t count) {
        const int64_t at = int64_t(t.ids.size());
        t.ids.insert(t.ids.end(), ids, ids + count);
        return at;
    }
    // One logical phase of rows: row r (output id first_row + r) sums the entries [ptr[r0 + r], ptr[r0 + r + 1]) of the
    // id list, which start at `at` in the pass's list and ascend within a row.  need(b, e) = the phase that must be
    // complete before the entries [b, e) may be read, or -1.  Rows longer than split.long_row are cut: their chunk
    // rows form a phase of their own, placed first, and the row itself becomes a short row over the chunks' partial rows.
    // Returns the index of the phase that holds the rows themselves.
    template <typename Need>
    int32_t rows_phase(const std::vector<int64_t> &ptr, int64_t r0, int64_t count, int32_t first_row, int64_t at, Need need) {
        const int64_t shift = at - ptr[r0];
        // entries of the pass's list in [b, e) that are not rows of the layer input (ids ascend within a row)
        auto n_sec_of = [&](int64_t b, int64_t e) {
            return int64_t((t.ids.data() + e) - std::lower_bound(t.ids.data() + b, t.ids.data() + e, n));
        };
        std::vector<int64_t> chunk_first;        // per long row: id of its first chunk row
        bool any_long = false;
        for (int64_t r = 0; r < count && !any_long; ++r) any_long = ptr[r0 + r + 1] - ptr[r0 + r] > split.long_row;
        int32_t chunk_phase = -1;
        if (any_long) {
            int64_t n_chunk_rows = 0;
            for (int64_t r = 0; r < count; ++r) {
                const int64_t len = ptr[r0 + r + 1] - ptr[r0 + r];
                if (len > split.long_row) n_chunk_rows += (len + split.chunk_len - 1) / split.chunk_len;
            }
            begin_phase(n_chunk_rows);
            chunk_phase = phase;
            for (int64_t r = 0; r < count; ++r) {
                const int64_t b = ptr[r0 + r], e = ptr[r0 + r + 1];
                if (e - b <= split.long_row) continue;
                chunk_first.push_back(int64_t(n) + k + t.n_chunks);
                for (int64_t cb = b; cb < e; cb += split.chunk_len) {
                    const int64_t ce = std::min<int64_t>(cb + split.chunk_len, e);
                    push_row(cb + shift, ce + shift, int32_t(int64_t(n) + k + t.n_chunks++), need(cb, ce), n_sec_of(cb + shift, ce + shift));
                }
            }
            end_phase();
        }
        begin_phase(count);
        size_t li = 0;
        for (int64_t r = 0; r < count; ++r) {
            const int64_t b = ptr[r0 + r], e = ptr[r0 + r + 1];
            if (e - b <= split.long_row) {
                push_row(b + shift, e + shift, int32_t(first_row + r), need(b, e), n_sec_of(b + shift, e + shift));
            } else {                             // the sum of its chunks' partial rows
                const int64_t n_chunk = (e - b + split.chunk_len - 1) / split.chunk_len;
                const int64_t eb = int64_t(t.ids.size());
                for (int64_t c = 0; c < n_chunk; ++c) t.ids.push_back(int32_t(chunk_first[li] + c));
                ++li;
                push_row(eb, eb + n_chunk, int32_t(first_row + r), chunk_phase, n_chunk);
            }
        }
        end_phase();
        return phase;
    }
    void finish() {
        t.last_phase = phase;
        t.ok = phase >= 0 && phase < kFusedMaxPhases && t.n_items() > 0 && t.n_items() < (int64_t(1) << 30) &&
               t.ids.size() < (size_t(1) << 31) && int64_t(n) + k + t.n_chunks < (int64_t(1) << 31);
        if (!t.ok) {
            t.items.clear();
            t.phase_size.clear();
            t.n_chunks = 0;
        }
    }
};

void build_fused(hag *h) {
    const int32_t n = h->n, k = h->num_agg, L = h->num_levels;
    std::vector<int32_t> clevel(k);
    for (int32_t l = 1; l <= L; ++l)
        for (int64_t j = h->level_ptr[l - 1]; j < h->level_ptr[l]; ++j) clevel[j] = l;
    auto level_of = [&](int32_t id) { return id < n ? 0 : clevel[id - n]; };
    std::vector<int32_t> phase_of_level(size_t(L) + 2, -1);      // phase that writes the rows of a level (forward: L + 1 = deeper than the cut)
    {   // forward over the HAG: levels 1..fwd_cut as rows of two entries, the expanded deeper nodes, the graph nodes
        const int32_t c = h->fwd_cut;
        const int64_t j0 = h->level_ptr[c];
        FusedBuilder fb(h->fz_fwd, n, k, fused_split_for_entries(h->e_res + int64_t(h->ftail_idx.size())));
        auto phase_of = [&](int32_t id) { const int32_t l = level_of(id); return l == 0 ? -1 : phase_of_level[l <= c ? l : c + 1]; };
        // ids ascend within a list and aggregation nodes are sorted by level: the last entry is written by the latest phase
        const std::vector<int32_t> *src = &h->agg_in;
        auto need = [&](int64_t b, int64_t e) { return e > b ? phase_of((*src)[e - 1]) : -1; };
        std::vector<int64_t> pair_ptr(size_t(j0) + 1);
        for (int64_t j = 0; j <= j0; ++j) pair_ptr[j] = 2 * j;
        const int64_t at_pairs = fb.add_ids(h->agg_in.data(), 2 * j0);
        for (int32_t l = 1; l <= c; ++l)
            phase_of_level[l] = fb.rows_phase(pair_ptr, h->level_ptr[l - 1], h->level_ptr[l] - h->level_ptr[l - 1],
                                              int32_t(n + h->level_ptr[l - 1]), at_pairs + 2 * h->level_ptr[l - 1], need);
        h->fz_fwd.off_head = fb.add_ids(h->ftail_idx.data(), int64_t(h->ftail_idx.size()));
        src = &h->ftail_idx;
        if (j0 < k) phase_of_level[c + 1] = fb.rows_phase(h->ftail_ptr, 0, k - j0, int32_t(n + j0), h->fz_fwd.off_head, need);
        h->fz_fwd.off_tail = fb.add_ids(h->res_idx.data(), h->e_res);
        src = &h->res_idx;
        const int64_t head = h->fz_fwd.n_items();
        if (n > 0) fb.rows_phase(h->res_ptr, 0, n, 0, h->fz_fwd.off_tail, need);
        fb.finish();
        h->fz_fwd.head_items = h->fz_fwd.ok ? head : 0;
    }
    {   // backward over the HAG: the expanded deep nodes, levels bwd_cut..1, the graph nodes as sources
        const int32_t c = h->bwd_cut;
        const int64_t j0 = h->level_ptr[c];
        FusedBuilder fb(h->fz_bwd, n, k, fused_split_for_entries(h->e_hat + int64_t(h->btail_idx.size())));
        std::fill(phase_of_level.begin(), phase_of_level.end(), -1);
        auto phase_of = [&](int32_t id) { const int32_t l = level_of(id); return l == 0 ? -1 : phase_of_level[l <= c ? l : c + 1]; };
        // destinations ascend: the first aggregation node among them is the shallowest, i.e. the one written by the latest phase
        auto need = [&](int64_t b, int64_t e) {
            const int32_t *lo = std::lower_bound(h->t_idx.data() + b, h->t_idx.data() + e, n);
            return lo < h->t_idx.data() + e ? phase_of(*lo) : -1;
        };
        h->fz_bwd.off_head = fb.add_ids(h->btail_idx.data(), int64_t(h->btail_idx.size()));
        if (j0 < k) phase_of_level[c + 1] = fb.rows_phase(h->btail_ptr, 0, k - j0, int32_t(n + j0), h->fz_bwd.off_head,
                                                          [](int64_t, int64_t) { return -1; });     // all sources are graph-node outputs
        h->fz_bwd.off_tail = fb.add_ids(h->t_idx.data(), h->e_hat);
        for (int32_t l = c; l >= 1; --l)
            phase_of_level[l] = fb.rows_phase(h->t_ptr, int64_t(n) + h->level_ptr[l - 1], h->level_ptr[l] - h->level_ptr[l - 1],
                                              int32_t(n + h->level_ptr[l - 1]), h->fz_bwd.off_tail + h->t_ptr[size_t(n) + h->level_ptr[l - 1]], need);
        const int64_t head = h->fz_bwd.n_items();
        if (n > 0) fb.rows_phase(h->t_ptr, 0, n, 0, h->fz_bwd.off_tail, need);
        fb.finish();
        h->fz_bwd.head_items = h->fz_bwd.ok ? head : 0;
    }
    {   // the input graph and its transpose: nothing to wait for but the chunks of long rows (k = 0: their ids start at n)
        auto none = [](int64_t, int64_t) { return -1; };
        FusedBuilder fb(h->fz_csr, n, 0, fused_split_for_entries(h->e));
        h->fz_csr.off_tail = fb.add_ids(h->csr_idx.data(), h->e);
        if (n > 0) fb.rows_phase(h->csr_ptr, 0, n, 0, 0, none);
        fb.finish();
        FusedBuilder ft(h->fz_csr_t, n, 0, fused_split_for_entries(h->e));
        h->fz_csr_t.off_tail = ft.add_ids(h->csr_t_idx.data(), h->e);
        if (n > 0) ft.rows_phase(h->csr_t_ptr, 0, n, 0, 0, none);
        ft.finish();
    }
    h->max_segs_hag = std::max(h->max_segs_hag, std::max(h->fz_fwd.n_chunks, h->fz_bwd.n_chunks));
    h->max_segs_csr = std::max(h->max_segs_csr, std::max(h->fz_csr.n_chunks, h->fz_csr_t.n_chunks));
}

}  // namespace

hag_status hag_layout(hag *h, const std::vector<int32_t> &rows_store, const std::vector<int32_t> &rows_len) {
    try {
        if (hag_alloc_should_fail(0)) throw std::bad_alloc();
        const int32_t n = h->n, k = h->num_agg;
        // level = 1 + the larger level of the two inputs (graph nodes are level 0)
        std::vector<int32_t> level(size_t(n) + k, 0);
        int32_t max_level = 0;
        for (int32_t j = 0; j < k; ++j) {
            const int32_t l = 1 + std::max(level[h->trace[3 * j]], level[h->trace[3 * j + 1]]);
            level[n + j] = l;
            max_level = std::max(max_level, l);
        }
        h->num_levels = max_level;
        h->level_ptr.assign(size_t(max_level) + 1, 0);
        for (int32_t j = 0; j < k; ++j) h->level_ptr[level[n + j]]++;
        // level_ptr[l] currently holds the size of level l (l >= 1); make it a running end
        for (int32_t l = 1; l <= max_level; ++l) h->level_ptr[l] += h->level_ptr[l - 1];
        // stable placement by (level, creation index)
        std::vector<int64_t> next(size_t(max_level) + 1, 0);
        for (int32_t l = 1; l <= max_level; ++l) next[l] = h->level_ptr[l - 1];
        std::vector<int32_t> canon(size_t(n) + k);
        for (int32_t v = 0; v < n; ++v) canon[v] = v;
        for (int32_t j = 0; j < k; ++j) canon[n + j] = int32_t(n + next[level[n + j]]++);
        h->agg_in.assign(size_t(2) * k, 0);
        for (int32_t j = 0; j < k; ++j) {
            const int32_t a = canon[h->trace[3 * j]], b = canon[h->trace[3 * j + 1]];
            const int32_t pos = canon[n + j] - n;
            h->agg_in[2 * pos] = std::min(a, b);
            h->agg_in[2 * pos + 1] = std::max(a, b);
        }
        // residual CSR in canonical ids, every row ascending
        h->res_ptr.assign(size_t(n) + 1, 0);
        for (int32_t v = 0; v < n; ++v) h->res_ptr[v + 1] = h->res_ptr[v] + rows_len[v];
        h->e_res = h->res_ptr[n];
        h->res_idx.resize(h->e_res);
        int32_t max_res = 0;
        for (int32_t v = 0; v < n; ++v) {
            const int32_t *src = rows_store.data() + h->csr_ptr[v];
            int32_t *dst = h->res_idx.data() + h->res_ptr[v];
            for (int32_t j = 0; j < rows_len[v]; ++j) dst[j] = canon[src[j]];
            std::sort(dst, dst + rows_len[v]);
            max_res = std::max(max_res, rows_len[v]);
        }
        h->e_hat = h->e_res + 2 * int64_t(k);
        // transposed HAG by counting sort; destinations come out ascending because
        // graph-node rows are visited first in id order, then aggregation nodes in id order
        const size_t n_src = size_t(n) + k;
        h->t_ptr.assign(n_src + 1, 0);
        for (int64_t i = 0; i < h->e_res; ++i) h->t_ptr[h->res_idx[i] + 1]++;
        for (int64_t i = 0; i < 2 * int64_t(k); ++i) h->t_ptr[h->agg_in[i] + 1]++;
        int64_t max_out = 0;
        for (size_t s = 0; s < n_src; ++s) {
            max_out = std::max(max_out, h->t_ptr[s + 1]);
            h->t_ptr[s + 1] += h->t_ptr[s];
        }
        h->t_idx.resize(h->e_hat);
        {
            std::vector<int64_t> fill(h->t_ptr.begin(), h->t_ptr.end() - 1);
            for (int32_t v = 0; v < n; ++v)
                for (int64_t i = h->res_ptr[v]; i < h->res_ptr[v + 1]; ++i) h->t_idx[fill[h->res_idx[i]]++] = v;
            for (int32_t j = 0; j < k; ++j) {
                h->t_idx[fill[h->agg_in[2 * j]]++] = n + j;
                h->t_idx[fill[h->agg_in[2 * j + 1]]++] = n + j;
            }
        }
        // transposed input graph, same method
        h->csr_t_ptr.assign(size_t(n) + 1, 0);
        for (int64_t i = 0; i < h->e; ++i) h->csr_t_ptr[h->csr_idx[i] + 1]++;
        for (int32_t s = 0; s < n; ++s) h->csr_t_ptr[s + 1] += h->csr_t_ptr[s];
        h->csr_t_idx.resize(h->e);
        {
            std::vector<int64_t> fill(h->csr_t_ptr.begin(), h->csr_t_ptr.end() - 1);
            for (int32_t v = 0; v < n; ++v)
                for (int64_t i = h->csr_ptr[v]; i < h->csr_ptr[v + 1]; ++i) h->csr_t_idx[fill[h->csr_idx[i]]++] = v;
        }
        int32_t fwd_cut = 0, bwd_cut = 0;
        choose_cuts(h, fwd_cut, bwd_cut);
        expand_tails(h, fwd_cut, bwd_cut);
        build_segments(h);
        build_fused(h);
        // counters of the cost function
        hag_info &f = h->info;
        f = hag_info{};
        f.n = n;
        f.capacity = h->capacity;
        f.num_agg = k;
        f.num_levels = max_level;
        f.e = h->e;
        f.e_hat = h->e_hat;
        int32_t max_in = 0;
        for (int32_t v = 0; v < n; ++v) {
            const int32_t deg = h->in_degree[v];
            max_in = std::max(max_in, deg);
            f.aggregations_gnn += std::max(deg - 1, 0);
            f.aggregations_hag += std::max(rows_len[v] - 1, 0);
        }
        f.aggregations_hag += k;  // two in-edges each: one binary aggregation
        f.aggregations_hag_closed = h->e_hat - n - k;
        for (int32_t j = 0; j < k; ++j) f.saved += h->trace[3 * j + 2] - 1;
        f.first_redundancy = k ? h->trace[2] : 0;
        f.last_redundancy = k ? h->trace[3 * (k - 1) + 2] : 0;
        f.max_in_degree = max_in;
        f.max_res_degree = max_res;
        f.max_out_degree = int32_t(max_out);
        f.device = -1;
    } catch (const std::bad_alloc &) {
        return HAG_ERR_OOM_HOST;
    }
    return HAG_OK;
}

extern "C" hag_status hag_build(int32_t n, const int64_t *row_ptr, const int32_t *col_idx, int32_t capacity, hag_t **out) {
    return hag_build_ex(n, row_ptr, col_idx, capacity, 2, out);
}

namespace {

// Argument and graph checks shared by hag_build_ex and hag_import; nothing reads through the CSR before they pass.
hag_status validate_graph(int32_t n, const int64_t *row_ptr, const int32_t *col_idx, int64_t capacity) {
    if (!row_ptr || (!col_idx && n > 0 && row_ptr[n] > 0)) return HAG_ERR_NULL;
    if (n < 0 || capacity < 0) return HAG_ERR_ARG;
    if (int64_t(n) + capacity >= (int64_t(1) << 31)) return HAG_ERR_ARG;
    if (row_ptr[0] != 0) return HAG_ERR_GRAPH;
    for (int32_t v = 0; v < n; ++v)
        if (row_ptr[v + 1] < row_ptr[v]) return HAG_ERR_GRAPH;
    if (row_ptr[n] >= (int64_t(1) << 31)) return HAG_ERR_ARG;
    for (int32_t v = 0; v < n; ++v) {
        int64_t prev = -1;
        for (int64_t i = row_ptr[v]; i < row_ptr[v + 1]; ++i) {
            const int64_t c = col_idx[i];
            if (c < 0 || c >= n || c <= prev) return HAG_ERR_GRAPH;
            prev = c;
        }
    }
    return HAG_OK;
}

// Builds a handle from the graph and either the search (trace == nullptr) or a recorded trace of num_merges merges.
hag_status build_handle(int32_t n, const int64_t *row_ptr, const int32_t *col_idx, int32_t capacity, int32_t min_redundancy,
                        const int32_t *trace, int32_t num_merges, hag_t **out) {
    const auto t0 = std::chrono::steady_clock::now();
    hag *h = new (std::nothrow) hag();
    if (!h) return HAG_ERR_OOM_HOST;
    hag_status st = HAG_OK;
    try {
        h->n = n;
        h->capacity = capacity;
        h->min_redundancy = min_redundancy;
        h->e = row_ptr[n];
        h->csr_ptr.assign(row_ptr, row_ptr + n + 1);
        h->csr_idx.assign(col_idx, col_idx + h->e);
        h->in_degree.resize(n);
        for (int32_t v = 0; v < n; ++v) h->in_degree[v] = int32_t(row_ptr[v + 1] - row_ptr[v]);
        std::vector<int32_t> rows_store, rows_len;
        if (!trace) {
            st = hag_search(h, rows_store, rows_len);
        } else {
            if (hag_alloc_should_fail(0)) throw std::bad_alloc();
            rows_store = h->csr_idx;
            rows_len.resize(n);
            for (int32_t u = 0; u < n; ++u) rows_len[u] = int32_t(h->csr_ptr[u + 1] - h->csr_ptr[u]);
            if (num_merges > 0) {
                const std::vector<int32_t> recorded(trace, trace + size_t(3) * num_merges);
                for (int32_t i = 0; i < num_merges; ++i)
                    if (recorded[3 * i + 2] < 2) st = HAG_ERR_ARG;           // not a merge Algorithm 3 would make
                if (st == HAG_OK) {
                    Searcher s(n, num_merges, h->csr_ptr.data(), rows_store, rows_len);
                    st = s.replay(recorded, num_merges, h->trace);
                }
            }
            h->num_agg = int32_t(h->trace.size() / 3);
        }
        if (st == HAG_OK) st = hag_layout(h, rows_store, rows_len);
    } catch (const std::bad_alloc &) {
        st = HAG_ERR_OOM_HOST;
    }
    if (st != HAG_OK) {
        delete h;
        return st;
    }
    h->info.build_seconds = std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count();
    *out = h;
    return HAG_OK;
}

}  // namespace

extern "C" hag_status hag_build_ex(int32_t n, const int64_t *row_ptr, const int32_t *col_idx, int32_t capacity,
                                   int32_t min_redundancy, hag_t **out) {
    if (!out) return HAG_ERR_NULL;
    *out = nullptr;
    if (min_redundancy < 2) return HAG_ERR_ARG;
    const hag_status st = validate_graph(n, row_ptr, col_idx, capacity);
    if (st != HAG_OK) return st;
    return build_handle(n, row_ptr, col_idx, capacity, min_redundancy, nullptr, 0, out);
}

extern "C" hag_status hag_import(int32_t n, const int64_t *row_ptr, const int32_t *col_idx, int32_t num_merges,
                                 const int32_t *trace, hag_t **out) {
    if (!out) return HAG_ERR_NULL;
    *out = nullptr;
    if (num_merges < 0) return HAG_ERR_ARG;
    if (num_merges > 0 && !trace) return HAG_ERR_NULL;
    const hag_status st = validate_graph(n, row_ptr, col_idx, num_merges);
    if (st != HAG_OK) return st;
    static const int32_t no_merges[3] = {0, 0, 0};          // (a non-null trace is what selects the replay)
    return build_handle(n, row_ptr, col_idx, num_merges, 2, trace ? trace : no_merges, num_merges, out);
}

extern "C" int32_t hag_build_threads(int32_t threads) {
    const int prev = g_build_threads.load();
    if (threads >= 0) g_build_threads.store(threads);
    return prev;
}

extern "C" hag_status hag_set_cuts(hag_t *h, int32_t fwd_cut, int32_t bwd_cut) {
    if (!h) return HAG_ERR_NULL;
    if (h->device >= 0) return HAG_ERR_ARG;                    // the device copy is made once
    if (fwd_cut < -1 || fwd_cut > h->num_levels || bwd_cut < -1 || bwd_cut > h->num_levels) return HAG_ERR_ARG;
    try {
        int32_t f = 0, b = 0;
        if (fwd_cut < 0 || bwd_cut < 0) choose_cuts(h, f, b);
        expand_tails(h, fwd_cut < 0 ? f : fwd_cut, bwd_cut < 0 ? b : bwd_cut);
        build_segments(h);
        build_fused(h);
    } catch (const std::bad_alloc &) {
        return HAG_ERR_OOM_HOST;
    }
    return HAG_OK;
}

extern "C" hag_status hag_truncate(const hag_t *src, int32_t capacity, hag_t **out) {
    if (!out) return HAG_ERR_NULL;
    *out = nullptr;
    if (!src) return HAG_ERR_NULL;
    if (capacity < 0) return HAG_ERR_ARG;
    // beyond the recorded merges the answer is known only if the search ended by itself
    if (capacity > src->num_agg && src->num_agg == src->capacity) return HAG_ERR_ARG;
    const auto t0 = std::chrono::steady_clock::now();
    hag *h = new (std::nothrow) hag();
    if (!h) return HAG_ERR_OOM_HOST;
    hag_status st = HAG_OK;
    try {
        const int32_t k = std::min(capacity, src->num_agg);
        h->n = src->n;
        h->capacity = capacity;
        h->min_redundancy = src->min_redundancy;
        h->e = src->e;
        h->csr_ptr = src->csr_ptr;
        h->csr_idx = src->csr_idx;
        h->in_degree = src->in_degree;
        std::vector<int32_t> rows_store = h->csr_idx, rows_len(h->n);
        for (int32_t u = 0; u < h->n; ++u) rows_len[u] = int32_t(h->csr_ptr[u + 1] - h->csr_ptr[u]);
        if (k > 0) {
            Searcher s(h->n, k, h->csr_ptr.data(), rows_store, rows_len);
            st = s.replay(src->trace, k, h->trace);
        }
        h->num_agg = int32_t(h->trace.size() / 3);
        if (st == HAG_OK) st = hag_layout(h, rows_store, rows_len);
    } catch (const std::bad_alloc &) {
        st = HAG_ERR_OOM_HOST;
    }
    if (st != HAG_OK) {
        delete h;
        return st;
    }
    h->info.build_seconds = std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count();
    *out = h;
    return HAG_OK;
}

extern "C" hag_status hag_get_info(const hag_t *h, hag_info *out) {
    if (!h || !out) return HAG_ERR_NULL;
    *out = h->info;
    out->device = h->device;
    return HAG_OK;
}

extern "C" hag_status hag_export(const hag_t *h, hag_arrays *out) {
    if (!h || !out) return HAG_ERR_NULL;
    out->n = h->n;
    out->num_agg = h->num_agg;
    out->num_levels = h->num_levels;
    out->level_ptr = h->level_ptr.data();
    out->agg_in = h->agg_in.data();
    out->res_ptr = h->res_ptr.data();
    out->res_idx = h->res_idx.data();
    out->t_ptr = h->t_ptr.data();
    out->t_idx = h->t_idx.data();
    out->in_degree = h->in_degree.data();
    out->trace = h->trace.data();
    out->csr_t_ptr = h->csr_t_ptr.data();
    out->csr_t_idx = h->csr_t_idx.data();
    out->fwd_cut = h->fwd_cut;
    out->bwd_cut = h->bwd_cut;
    out->ftail_ptr = h->ftail_ptr.data();
    out->ftail_idx = h->ftail_idx.data();
    out->btail_ptr = h->btail_ptr.data();
    out->btail_idx = h->btail_idx.data();
    return HAG_OK;
}

extern "C" hag_status hag_export_pass(const hag_t *h, int32_t pass, hag_pass_view *out) {
    if (!h || !out) return HAG_ERR_NULL;
    if (pass < 0 || pass > 3) return HAG_ERR_ARG;
    const fused_table &t = pass == 0 ? h->fz_fwd : (pass == 1 ? h->fz_bwd : (pass == 2 ? h->fz_csr : h->fz_csr_t));
    *out = hag_pass_view{};
    if (!t.ok) return HAG_OK;
    out->n_rows = t.n_items();
    out->n_phases = int64_t(t.phase_size.size());
    out->n_chunk_rows = t.n_chunks;
    out->n_ids = int64_t(t.ids.size());
    out->rows = t.items.data();
    out->phase_size = t.phase_size.data();
    out->ids = t.ids.data();
    return HAG_OK;
}

extern "C" hag_status hag_export_row_order(const hag_t *h, int32_t list, int32_t *first_row, int64_t *count, const int32_t **order) {
    if (!h || !first_row || !count || !order) return HAG_ERR_NULL;
    if (list < 0 || list > 5) return HAG_ERR_ARG;
    const seg_set *sets[6] = {&h->seg_res, &h->seg_t, &h->seg_csr, &h->seg_csr_t, &h->seg_ftail, &h->seg_btail};
    *first_row = sets[list]->order_first_row;
    *count = int64_t(sets[list]->order.size());
    *order = sets[list]->order.empty() ? nullptr : sets[list]->order.data();
    return HAG_OK;
}

extern "C" int32_t hag_test_range_predicates(int32_t id, int32_t lo, int32_t hi, int64_t i, int64_t rows, int32_t prev, int32_t cur,
                                              int32_t first, int32_t last) {
    return (hag_id_in_range(id, lo, hi) ? 1 : 0) | (hag_ptr_ok(i, rows, prev, cur, first, last) ? 2 : 0);
}

extern "C" const char *hag_status_str(hag_status s) {
    switch (s) {
        case HAG_OK: return "ok";
        case HAG_ERR_NULL: return "null pointer";
        case HAG_ERR_ARG: return "argument out of range";
        case HAG_ERR_GRAPH: return "malformed graph (rows must be strictly ascending, ids in range)";
        case HAG_ERR_OOM_HOST: return "out of host memory";
        case HAG_ERR_OOM_DEVICE: return "out of device memory";
        case HAG_ERR_CUDA: return "CUDA runtime error";
        case HAG_ERR_DTYPE: return "unsupported dtype";
        case HAG_ERR_ALIGN: return "pointer or row size not 16-byte aligned";
        case HAG_ERR_WORKSPACE: return "workspace required but missing";
        case HAG_ERR_TIMEOUT: return "device-side wait timed out";
        case HAG_ERR_NOT_ON_DEVICE: return "structure not on a device (call hag_to_device)";
        case HAG_ERR_TOO_LARGE: return "aggregation-node rows exceed the built-in scratch array (HAG_STATIC_SCRATCH_BYTES)";
    }
    return "unknown status";
}
