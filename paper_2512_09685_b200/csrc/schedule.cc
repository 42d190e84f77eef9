// Host-side group-schedule encoder: synchronization-mode decision -> CSR pair.
// No CUDA call in this file.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <vector>

#include "star.h"

namespace {

bool workers_distinct_in_range(const int32_t *workers, int count, int W)
{
    uint64_t seen = 0;                       // W <= STAR_MAX_WORKERS == 64
    for (int j = 0; j < count; ++j) {
        const int32_t w = workers[j];
        if (w < 0 || w >= W) return false;
        if (seen >> w & 1u) return false;
        seen |= uint64_t{1} << w;
    }
    return true;
}

// Writes the groups (each a list of workers) as CSR.
void pack(const std::vector<std::vector<int32_t>> &groups, int32_t *offsets_out, int32_t *members_out,
          int *n_groups_out)
{
    int32_t pos = 0;
    offsets_out[0] = 0;
    for (size_t k = 0; k < groups.size(); ++k) {
        for (int32_t w : groups[k]) members_out[pos++] = w;
        offsets_out[k + 1] = pos;
    }
    *n_groups_out = static_cast<int>(groups.size());
}

}  // namespace

extern "C" star_status_t star_schedule_validate(const int32_t *group_offsets, const int32_t *group_members,
                                                int n_groups, int W)
{
    if (n_groups < 0 || W < 0) return STAR_ERR_INVALID_ARG;
    if (W > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    if (n_groups == 0) return STAR_OK;
    if (!group_offsets || !group_members) return STAR_ERR_NULL_POINTER;
    if (n_groups > W || group_offsets[0] != 0) return STAR_ERR_BAD_SCHEDULE;
    for (int k = 0; k < n_groups; ++k) {
        if (group_offsets[k + 1] <= group_offsets[k]) return STAR_ERR_BAD_SCHEDULE;   // empty group
        if (group_offsets[k + 1] > W) return STAR_ERR_BAD_SCHEDULE;                   // > W members in total
    }
    if (!workers_distinct_in_range(group_members, group_offsets[n_groups], W)) return STAR_ERR_BAD_SCHEDULE;
    return STAR_OK;
}

extern "C" star_status_t star_schedule_static_x(const int32_t *arrival_order, int n_arrived, int W, int x,
                                                int sort_members, int32_t *offsets_out,
                                                int32_t *members_out, int *n_groups_out)
{
    if (!offsets_out || !members_out || !n_groups_out) return STAR_ERR_NULL_POINTER;
    if (W < 0 || x < 1) return STAR_ERR_INVALID_ARG;
    if (W > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    std::vector<int32_t> order;
    if (arrival_order) {
        if (n_arrived < 0 || n_arrived > W) return STAR_ERR_INVALID_ARG;
        if (!workers_distinct_in_range(arrival_order, n_arrived, W)) return STAR_ERR_BAD_SCHEDULE;
        order.assign(arrival_order, arrival_order + n_arrived);
    } else {
        if (n_arrived != W) return STAR_ERR_INVALID_ARG;
        order.resize(W);
        for (int w = 0; w < W; ++w) order[w] = w;
    }
    std::vector<std::vector<int32_t>> groups;
    for (size_t start = 0; start < order.size(); start += static_cast<size_t>(x)) {
        const size_t stop = std::min(order.size(), start + static_cast<size_t>(x));
        std::vector<int32_t> g(order.begin() + start, order.begin() + stop);
        if (sort_members) std::sort(g.begin(), g.end());
        groups.push_back(std::move(g));
    }
    pack(groups, offsets_out, members_out, n_groups_out);
    return STAR_OK;
}

namespace {

// Workers grouped by label, groups in ascending label order, members ascending.
star_status_t groups_by_label(const int32_t *label, int W, std::vector<std::vector<int32_t>> *groups)
{
    if (W < 0) return STAR_ERR_INVALID_ARG;
    if (W > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    std::vector<int32_t> distinct;
    for (int w = 0; w < W; ++w) {
        if (label[w] < -1) return STAR_ERR_INVALID_ARG;
        if (label[w] >= 0) distinct.push_back(label[w]);
    }
    std::sort(distinct.begin(), distinct.end());
    distinct.erase(std::unique(distinct.begin(), distinct.end()), distinct.end());
    groups->assign(distinct.size(), {});
    for (int w = 0; w < W; ++w) {
        if (label[w] < 0) continue;
        const size_t k = std::lower_bound(distinct.begin(), distinct.end(), label[w]) - distinct.begin();
        (*groups)[k].push_back(w);
    }
    return STAR_OK;
}

}  // namespace

extern "C" star_status_t star_schedule_from_labels(const int32_t *group_of_worker, int W,
                                                   int32_t *offsets_out, int32_t *members_out,
                                                   int *n_groups_out)
{
    if (!offsets_out || !members_out || !n_groups_out) return STAR_ERR_NULL_POINTER;
    if (!group_of_worker && W > 0) return STAR_ERR_NULL_POINTER;
    std::vector<std::vector<int32_t>> groups;
    const star_status_t st = groups_by_label(group_of_worker, W, &groups);
    if (st != STAR_OK) return st;
    pack(groups, offsets_out, members_out, n_groups_out);
    return STAR_OK;
}

extern "C" star_status_t star_schedule_dynamic_x(const double *iter_time, const int32_t *cluster_of_worker,
                                                 int W, int32_t *offsets_out, int32_t *members_out,
                                                 int *n_groups_out)
{
    if (!offsets_out || !members_out || !n_groups_out) return STAR_ERR_NULL_POINTER;
    if ((!iter_time || !cluster_of_worker) && W > 0) return STAR_ERR_NULL_POINTER;
    std::vector<std::vector<int32_t>> clusters;
    const star_status_t st = groups_by_label(cluster_of_worker, W, &clusters);
    if (st != STAR_OK) return st;
    for (int w = 0; w < W; ++w)
        if (cluster_of_worker[w] >= 0 && !std::isfinite(iter_time[w])) return STAR_ERR_INVALID_ARG;
    // t_c = the slowest member's iteration time; clusters ascending in t_c.
    std::vector<double> slowest(clusters.size());
    for (size_t c = 0; c < clusters.size(); ++c) {
        double t = iter_time[clusters[c][0]];
        for (int32_t w : clusters[c]) t = std::max(t, iter_time[w]);
        slowest[c] = t;
    }
    std::vector<size_t> order(clusters.size());
    for (size_t c = 0; c < order.size(); ++c) order[c] = c;
    std::sort(order.begin(), order.end(), [&](size_t a, size_t b) {
        if (slowest[a] != slowest[b]) return slowest[a] < slowest[b];
        return clusters[a][0] < clusters[b][0];
    });
    std::vector<std::vector<int32_t>> groups;
    for (size_t c : order) groups.push_back(clusters[c]);
    pack(groups, offsets_out, members_out, n_groups_out);
    return STAR_OK;
}

extern "C" star_status_t star_shard_range(int64_t n, int world, int rank, int64_t align,
                                          int64_t *first_out, int64_t *count_out)
{
    if (!first_out || !count_out) return STAR_ERR_NULL_POINTER;
    if (n < 0 || world < 1 || rank < 0 || rank >= world || align < 1) return STAR_ERR_INVALID_ARG;
    // Split the ceil(n / align) blocks of `align` elements as evenly as possible;
    // the last block may be partial.
    const int64_t blocks = (n + align - 1) / align;
    const int64_t base = blocks / world, extra = blocks % world;
    const int64_t first_block = base * rank + (rank < extra ? rank : extra);
    const int64_t n_blocks = base + (rank < extra ? 1 : 0);
    int64_t first = first_block * align, last = (first_block + n_blocks) * align;
    if (first > n) first = n;
    if (last > n) last = n;
    *first_out = first;
    *count_out = last - first;
    return STAR_OK;
}
