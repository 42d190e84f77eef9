// Host-side mode decision: cluster the workers' predicted iteration times,
// evaluate the paper's time-to-progress estimates (Section IV-C1, Eq. 1 and
// Eq. 2) and emit the schedule of the cheapest mode.  No CUDA call here.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <vector>

#include "star.h"

namespace {

bool times_ok(const double *t, int W)
{
    for (int w = 0; w < W; ++w)
        if (!std::isfinite(t[w]) || t[w] <= 0.0) return false;
    return true;
}

// Mean of |t_i - t_j| over i in a, j in b (members ascending, a-major order).
double average_distance(const double *t, const std::vector<int> &a, const std::vector<int> &b)
{
    double sum = 0.0;
    for (int i : a)
        for (int j : b) sum += std::fabs(t[i] - t[j]);
    return sum / static_cast<double>(a.size() * b.size());
}

}  // namespace

extern "C" star_status_t star_cluster_iteration_times(const double *iter_time, int W, int n_clusters,
                                                      double max_distance, int32_t *cluster_of_worker_out,
                                                      int *n_clusters_out)
{
    if (!n_clusters_out || (W > 0 && (!iter_time || !cluster_of_worker_out))) return STAR_ERR_NULL_POINTER;
    if (W < 0 || std::isnan(max_distance)) return STAR_ERR_INVALID_ARG;
    if (W > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    if (!times_ok(iter_time, W)) return STAR_ERR_INVALID_ARG;
    // Clusters are kept ordered by their smallest member, members ascending.
    std::vector<std::vector<int>> clusters(W);
    for (int w = 0; w < W; ++w) clusters[w] = {w};
    const size_t want = n_clusters > 0 ? static_cast<size_t>(n_clusters) : 1;
    while (clusters.size() > want) {
        size_t best_a = 0, best_b = 1;
        double best = average_distance(iter_time, clusters[0], clusters[1]);
        for (size_t a = 0; a < clusters.size(); ++a)
            for (size_t b = a + 1; b < clusters.size(); ++b) {
                const double d = average_distance(iter_time, clusters[a], clusters[b]);
                if (d < best) {            // strict: ties keep the pair with the smaller leading members
                    best = d;
                    best_a = a;
                    best_b = b;
                }
            }
        if (max_distance >= 0.0 && best > max_distance) break;
        std::vector<int> merged;
        std::merge(clusters[best_a].begin(), clusters[best_a].end(), clusters[best_b].begin(),
                   clusters[best_b].end(), std::back_inserter(merged));
        clusters[best_a] = std::move(merged);           // keeps the smaller leading member: order is preserved
        clusters.erase(clusters.begin() + static_cast<std::ptrdiff_t>(best_b));
    }
    for (size_t c = 0; c < clusters.size(); ++c)
        for (int w : clusters[c]) cluster_of_worker_out[w] = static_cast<int32_t>(c);
    *n_clusters_out = static_cast<int>(clusters.size());
    return STAR_OK;
}

extern "C" star_status_t star_mode_times(const double *iter_time, const int32_t *cluster_of_worker, int W,
                                         double phi, double M, double *T_static_out, double *T_dynamic_out)
{
    if (!iter_time || !T_static_out) return STAR_ERR_NULL_POINTER;
    if (cluster_of_worker && !T_dynamic_out) return STAR_ERR_NULL_POINTER;
    if (W < 1 || !(phi >= 0.0) || !(M > 0.0) || !std::isfinite(phi) || !std::isfinite(M)) return STAR_ERR_INVALID_ARG;
    if (W > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    if (!times_ok(iter_time, W)) return STAR_ERR_INVALID_ARG;
    const double N = static_cast<double>(W);
    // Eq. 1 with t_x = the x-th smallest predicted iteration time.
    std::vector<double> sorted(iter_time, iter_time + W);
    std::sort(sorted.begin(), sorted.end());
    for (int x = 1; x <= W; ++x)
        T_static_out[x - 1] = (1.0 + phi / (static_cast<double>(x) * M / N)) * sorted[x - 1];
    if (!cluster_of_worker) return STAR_OK;
    // Eq. 2 over the clusters in ascending id.
    std::vector<int32_t> ids;
    for (int w = 0; w < W; ++w) {
        if (cluster_of_worker[w] < 0) return STAR_ERR_INVALID_ARG;      // every worker belongs to a cluster
        ids.push_back(cluster_of_worker[w]);
    }
    std::sort(ids.begin(), ids.end());
    ids.erase(std::unique(ids.begin(), ids.end()), ids.end());
    double total = 0.0;
    for (int32_t c : ids) {
        int n_c = 0;
        double t_c = 0.0;
        for (int w = 0; w < W; ++w)
            if (cluster_of_worker[w] == c) {
                t_c = n_c == 0 ? iter_time[w] : std::max(t_c, iter_time[w]);
                ++n_c;
            }
        total += 1.0 / ((1.0 + phi / (static_cast<double>(n_c) * M / N)) * t_c);
    }
    *T_dynamic_out = 1.0 / total;
    return STAR_OK;
}

extern "C" star_status_t star_choose_mode(const double *iter_time, const int32_t *cluster_of_worker, int W,
                                          double phi, double M, int *x_out, double *T_out,
                                          int32_t *offsets_out, int32_t *members_out, int *n_groups_out)
{
    if (!x_out || !T_out || !offsets_out || !members_out || !n_groups_out) return STAR_ERR_NULL_POINTER;
    if (W < 1) return STAR_ERR_INVALID_ARG;
    if (W > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    std::vector<double> T_static(W);
    double T_dynamic = 0.0;
    const star_status_t st = star_mode_times(iter_time, cluster_of_worker, W, phi, M, T_static.data(), &T_dynamic);
    if (st != STAR_OK) return st;
    int best_x = W;                                      // ties: the more synchronous mode
    double best_T = T_static[W - 1];
    for (int x = W - 1; x >= 1; --x)
        if (T_static[x - 1] < best_T) {
            best_x = x;
            best_T = T_static[x - 1];
        }
    if (cluster_of_worker && T_dynamic < best_T) {
        best_x = 0;
        best_T = T_dynamic;
    }
    *x_out = best_x;
    *T_out = best_T;
    if (best_x == 0) return star_schedule_dynamic_x(iter_time, cluster_of_worker, W, offsets_out, members_out, n_groups_out);
    // Static x-order: reports arrive in ascending predicted time (ties by index).
    std::vector<int32_t> order(W);
    for (int w = 0; w < W; ++w) order[w] = w;
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return iter_time[a] < iter_time[b]; });
    return star_schedule_static_x(order.data(), W, W, best_x, 1, offsets_out, members_out, n_groups_out);
}

// ---------------------------------------------------------------------------
// All-reduce architecture: which stragglers leave the ring and how long the
// parents wait (Section IV-C1, Eq. 3).
// ---------------------------------------------------------------------------
extern "C" star_status_t star_choose_all_reduce_mode(const double *iter_time, const double *child_time, int W,
                                                     double phi, double M, double t_w_max,
                                                     double straggler_threshold, int *x_out, double *t_w_out,
                                                     double *T_out, int32_t *removed_out, int32_t *offsets_out,
                                                     int32_t *members_out, int *n_groups_out)
{
    if (!iter_time || !child_time || !x_out || !t_w_out || !T_out || !removed_out || !offsets_out || !members_out ||
        !n_groups_out)
        return STAR_ERR_NULL_POINTER;
    if (W < 1 || !(phi >= 0.0) || !(M > 0.0) || !(t_w_max >= 0.0) || !(straggler_threshold >= 0.0) ||
        !std::isfinite(phi) || !std::isfinite(M) || !std::isfinite(t_w_max))
        return STAR_ERR_INVALID_ARG;
    if (W > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    if (!times_ok(iter_time, W) || !times_ok(child_time, W)) return STAR_ERR_INVALID_ARG;
    const double N = static_cast<double>(W);

    // Stragglers (Section II: deviation ratio above the threshold), slowest first.
    const double fastest = *std::min_element(iter_time, iter_time + W);
    std::vector<int32_t> slow;
    for (int w = 0; w < W; ++w)
        if ((iter_time[w] - fastest) / fastest > straggler_threshold) slow.push_back(w);
    std::sort(slow.begin(), slow.end(), [&](int32_t a, int32_t b) {
        if (iter_time[a] != iter_time[b]) return iter_time[a] > iter_time[b];
        return a > b;
    });

    bool have = false;
    int best_x = 0;
    double best_wait = 0.0, best_T = 0.0;
    const int max_removed = std::min<int>(static_cast<int>(slow.size()), W - 1);
    for (int x = 0; x <= max_removed; ++x) {
        std::vector<bool> is_removed(W, false);
        for (int j = 0; j < x; ++j) is_removed[slow[j]] = true;
        double t_ring = 0.0;
        for (int w = 0; w < W; ++w)
            if (!is_removed[w]) t_ring = std::max(t_ring, iter_time[w]);
        // Only t_w = 0 and the waits at which one more child makes it can be optimal.
        std::vector<double> waits{0.0};
        for (int j = 0; j < x; ++j) {
            const double need = child_time[slow[j]] - t_ring;
            if (need > 0.0 && need <= t_w_max) waits.push_back(need);
        }
        std::sort(waits.begin(), waits.end());
        waits.erase(std::unique(waits.begin(), waits.end()), waits.end());
        for (double t_w : waits) {
            int q = 0;
            for (int j = 0; j < x; ++j)
                if (child_time[slow[j]] - t_ring <= t_w) ++q;      // the form the candidate waits are built in
            const double T = (1.0 + phi / (static_cast<double>(W - x + q) * M / N)) * (t_ring + t_w);
            if (!have || T < best_T) {          // strict: ties keep fewer removals, then the shorter wait
                have = true;
                best_x = x;
                best_wait = t_w;
                best_T = T;
            }
        }
    }
    *x_out = best_x;
    *t_w_out = best_wait;
    *T_out = best_T;
    std::vector<bool> is_removed(W, false);
    for (int j = 0; j < best_x; ++j) {
        removed_out[j] = slow[j];
        is_removed[slow[j]] = true;
    }
    double t_ring = 0.0;
    for (int w = 0; w < W; ++w)
        if (!is_removed[w]) t_ring = std::max(t_ring, iter_time[w]);
    // One group: the ring members and the children whose reports are in on time.
    int32_t count = 0;
    for (int w = 0; w < W; ++w)
        if (!is_removed[w] || child_time[w] - t_ring <= best_wait) members_out[count++] = w;
    offsets_out[0] = 0;
    offsets_out[1] = count;
    *n_groups_out = 1;
    return STAR_OK;
}

// Parents of the removed workers: the j-th removed worker (as listed, slowest
// first) goes to ring member j mod R of the ring in ascending worker index.
extern "C" star_status_t star_assign_parents(const int32_t *removed, int x, int W, int32_t *parent_of_out)
{
    if (!parent_of_out || (x > 0 && !removed)) return STAR_ERR_NULL_POINTER;
    if (W < 1 || x < 0 || x >= W) return STAR_ERR_INVALID_ARG;
    if (W > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    std::vector<bool> is_removed(W, false);
    for (int j = 0; j < x; ++j) {
        if (removed[j] < 0 || removed[j] >= W || is_removed[removed[j]]) return STAR_ERR_INVALID_ARG;
        is_removed[removed[j]] = true;
    }
    std::vector<int32_t> ring;
    for (int w = 0; w < W; ++w)
        if (!is_removed[w]) ring.push_back(w);
    for (int w = 0; w < W; ++w) parent_of_out[w] = -1;
    for (int j = 0; j < x; ++j) parent_of_out[removed[j]] = ring[static_cast<size_t>(j) % ring.size()];
    return STAR_OK;
}

// Communication tree (Section IV-D2b): workers with longer latency sit lower.
// A fanout-ary tree filled layer by layer in ascending latency (ties: smaller
// index first): the `fanout` quickest workers are children of the root, the
// next `fanout` children of the quickest one, and so on.
extern "C" star_status_t star_build_tree(const double *latency, int W, int fanout, int32_t *parent_of_out)
{
    if (!parent_of_out || (W > 0 && !latency)) return STAR_ERR_NULL_POINTER;
    if (W < 0 || fanout < 1) return STAR_ERR_INVALID_ARG;
    if (W > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    for (int w = 0; w < W; ++w)
        if (!std::isfinite(latency[w])) return STAR_ERR_INVALID_ARG;
    std::vector<int32_t> order(W);
    for (int w = 0; w < W; ++w) order[w] = w;
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return latency[a] < latency[b]; });
    for (int i = 0; i < W; ++i)
        parent_of_out[order[i]] = i < fanout ? -1 : order[(i - fanout) / fanout];
    return STAR_OK;
}

