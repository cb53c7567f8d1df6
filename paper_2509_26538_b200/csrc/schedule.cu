// Host-side work lists and static schedules shared by the tensor-core kernels.
//
// A work item is a run of consecutive physical rows that share one list of up to three
// contiguous ranges (prefix, tile range, wrapped tile range -- or the whole sequence for
// prefix rows).  The forward kernel keeps the rows resident as queries and streams the
// ranges as keys; the backward kernels use the same lists in both directions, because the
// mask is symmetric (Sec. 3.2 / 3.3).  Every (item, batch * head) unit is assigned to a CTA on
// the host, longest units first onto the least-loaded CTA, and stored grouped by CTA.
#include <algorithm>
#include <functional>
#include <queue>
#include <utility>

#include "common.cuh"

namespace hilberta {

static void add_items(std::vector<WorkItem> &items, int row0, int rows, int item_rows, int block, int n_seg,
                      const int *seg_start, const int *seg_len) {
    for (int r = 0; r < rows; r += item_rows) {
        WorkItem it{};
        it.q_start = row0 + r;
        it.q_rows = std::min(item_rows, rows - r);
        it.n_seg = 0;
        it.kv_blocks = 0;
        for (int s = 0; s < n_seg; ++s) {
            if (seg_len[s] <= 0) continue;
            it.seg_start[it.n_seg] = seg_start[s];
            it.seg_len[it.n_seg] = seg_len[s];
            it.kv_blocks += (seg_len[s] + block - 1) / block;
            ++it.n_seg;
        }
        items.push_back(it);
    }
}

// Prefix rows see the whole sequence; the rows of each slid tile see the prefix and the
// tile's own one or two ranges.  item_rows: resident rows per item; block: streamed rows per
// block (kv_blocks counts them).
std::vector<WorkItem> build_work_items(const hilberta_plan_t *p, int item_rows, int block) {
    std::vector<WorkItem> items;
    {
        const int st[1] = {0}, ln[1] = {p->S};
        add_items(items, 0, p->P, item_rows, block, 1, st, ln);
    }
    for (const Window &w : p->h_windows) {
        const int st[3] = {0, w.seg0_start, w.seg1_start};
        const int ln[3] = {p->P, w.seg0_len, w.seg1_len};
        if (w.seg0_len > 0) add_items(items, w.seg0_start, w.seg0_len, item_rows, block, 3, st, ln);
        if (w.seg1_len > 0) add_items(items, w.seg1_start, w.seg1_len, item_rows, block, 3, st, ln);
    }
    return items;
}

// Every kernel reads the key ranges and query rows of its work items without further checks, so the
// lists are validated on the host before anything is uploaded: each item's rows and key ranges lie
// inside [0, S), its key ranges do not overlap, its block count matches them, and the items' query
// ranges cover [0, S) exactly once.
int check_work_items(const WorkItem *items, int n, int S, int item_rows, int block) {
    if (n < 0 || S < 0 || item_rows < 1 || block < 1 || (n > 0 && !items)) return HILBERTA_ERR_INVALID;
    std::vector<std::pair<int, int>> rows;   // (q_start, q_rows)
    rows.reserve((size_t)n);
    for (int i = 0; i < n; ++i) {
        const WorkItem &it = items[i];
        if (it.q_rows < 1 || it.q_rows > item_rows || it.q_start < 0 || it.q_start > S - it.q_rows)
            return HILBERTA_ERR_INVALID;
        if (it.n_seg < 1 || it.n_seg > 3) return HILBERTA_ERR_INVALID;
        long long blocks = 0;
        for (int a = 0; a < it.n_seg; ++a) {
            if (it.seg_len[a] < 1 || it.seg_start[a] < 0 || it.seg_start[a] > S - it.seg_len[a])
                return HILBERTA_ERR_INVALID;
            blocks += (it.seg_len[a] + block - 1) / block;
            for (int b = 0; b < a; ++b)
                if (it.seg_start[a] < it.seg_start[b] + it.seg_len[b] && it.seg_start[b] < it.seg_start[a] + it.seg_len[a])
                    return HILBERTA_ERR_INVALID;   // a key would be counted twice
        }
        if (blocks != it.kv_blocks) return HILBERTA_ERR_INVALID;
        rows.push_back(std::make_pair(it.q_start, it.q_rows));
    }
    std::sort(rows.begin(), rows.end());
    int next = 0;
    for (const std::pair<int, int> &r : rows) {
        if (r.first != next) return HILBERTA_ERR_INVALID;   // a gap or an overlap between items
        next = r.first + r.second;
    }
    return next == S ? HILBERTA_OK : HILBERTA_ERR_INVALID;
}

// The static schedule on the host: every (item, batch * head) unit -- items with a two-head cost as
// units of two consecutive indices -- goes, longest first, to the CTA with the smallest load so far.
// units: grouped by CTA; cta_begin: n_cta + 1 offsets.  Returns the largest CTA load.
long long build_schedule(int n_items, const long long *cost, const long long *cost_two_heads, int bh, int sm_count,
                         std::vector<WorkUnit> &units, std::vector<int> &cta_begin) {
    struct Costed {
        WorkUnit unit;
        long long cost;
    };
    std::vector<Costed> all;
    all.reserve((size_t)n_items * (size_t)bh);
    for (int i = 0; i < n_items; ++i) {
        const long long two = cost_two_heads ? cost_two_heads[i] : 0;
        int j = 0;
        if (two > 0)
            for (; j + 1 < bh; j += 2) all.push_back(Costed{WorkUnit{i, j, j + 1}, two});
        for (; j < bh; ++j) all.push_back(Costed{WorkUnit{i, j, -1}, cost[i]});
    }
    // paired units may cost more than the single units of an earlier item, hence the sort (stable:
    // equal costs keep the order of the items and of the heads)
    std::stable_sort(all.begin(), all.end(), [](const Costed &a, const Costed &b) { return a.cost > b.cost; });
    const long long n_units = (long long)all.size();
    const int n_cta = (int)std::min<long long>(n_units, sm_count);
    std::vector<std::vector<WorkUnit>> bins((size_t)std::max(n_cta, 0));
    typedef std::pair<long long, int> Load;  // (load, cta)
    std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
    for (int c = 0; c < n_cta; ++c) heap.push(Load(0, c));
    long long makespan = 0;
    for (const Costed &cu : all) {
        Load top = heap.top();
        heap.pop();
        bins[top.second].push_back(cu.unit);
        heap.push(Load(top.first + cu.cost, top.second));
        makespan = std::max(makespan, top.first + cu.cost);
    }
    units.clear();
    units.reserve((size_t)n_units);
    cta_begin.assign((size_t)n_cta + 1, 0);
    for (int c = 0; c < n_cta; ++c) {
        cta_begin[c] = (int)units.size();
        units.insert(units.end(), bins[c].begin(), bins[c].end());
    }
    cta_begin[n_cta] = (int)units.size();
    return makespan;
}

// items must be sorted by descending cost.  On success *d_units holds the units grouped by CTA and
// *d_cta_begin the n_cta + 1 offsets (both device memory, owned by the caller).
int upload_schedule(const std::vector<WorkItem> &items, const std::vector<long long> &cost, int bh, int sm_count,
                    WorkUnit **d_units, int **d_cta_begin, int *n_cta_out, const std::vector<long long> *cost_two_heads) {
    if ((long long)items.size() * bh > (1ll << 30)) return HILBERTA_ERR_INVALID;
    std::vector<WorkUnit> units;
    std::vector<int> cta_begin;
    build_schedule((int)items.size(), cost.data(), cost_two_heads ? cost_two_heads->data() : nullptr, bh, sm_count, units,
                   cta_begin);
    *n_cta_out = (int)cta_begin.size() - 1;
    HB_CUDA(cudaMalloc(d_units, sizeof(WorkUnit) * units.size()));
    HB_CUDA(cudaMemcpy(*d_units, units.data(), sizeof(WorkUnit) * units.size(), cudaMemcpyHostToDevice));
    HB_CUDA(cudaMalloc(d_cta_begin, sizeof(int) * cta_begin.size()));
    HB_CUDA(cudaMemcpy(*d_cta_begin, cta_begin.data(), sizeof(int) * cta_begin.size(), cudaMemcpyHostToDevice));
    return HILBERTA_OK;
}

}  // namespace hilberta

static_assert(sizeof(hilberta::WorkItem) == 10 * sizeof(int32_t), "hilberta_check_work_list takes ten ints per item");

extern "C" int hilberta_check_work_list(const int32_t *items, int n_items, int S, int item_rows, int block) {
    return hilberta::check_work_items(reinterpret_cast<const hilberta::WorkItem *>(items), n_items, S, item_rows, block);
}

static_assert(sizeof(hilberta::WorkUnit) == 3 * sizeof(int32_t), "hilberta_schedule_units writes three ints per unit");

extern "C" int hilberta_schedule_units(int n_items, const int64_t *cost, const int64_t *cost_two_heads, int bh, int n_cta,
                                       int32_t *units, int32_t *cta_begin, int64_t *largest_load) {
    if (n_items < 0 || bh < 1 || n_cta < 1 || (n_items > 0 && !cost) || !units || !cta_begin) return HILBERTA_ERR_INVALID;
    if ((long long)n_items * bh > (1ll << 30)) return HILBERTA_ERR_INVALID;
    std::vector<long long> c1(cost, cost + n_items), c2;
    if (cost_two_heads) c2.assign(cost_two_heads, cost_two_heads + n_items);
    std::vector<hilberta::WorkUnit> u;
    std::vector<int> cb;
    const long long m = hilberta::build_schedule(n_items, c1.data(), cost_two_heads ? c2.data() : nullptr, bh, n_cta, u, cb);
    for (size_t i = 0; i < u.size(); ++i) {
        units[3 * i] = u[i].item;
        units[3 * i + 1] = u[i].bh;
        units[3 * i + 2] = u[i].bh2;
    }
    for (int c = 0; c <= n_cta; ++c) cta_begin[c] = c < (int)cb.size() ? cb[c] : (int)u.size();
    if (largest_load) *largest_load = m;
    return HILBERTA_OK;
}
