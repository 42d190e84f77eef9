/*
 * star.h — C ABI of the B200 grouped gradient aggregation + parameter update.
 *
 * The operation (STAR's parameter-server hot path).  A round hands the server W
 * workers' gradient buffers and a SCHEDULE: an ordered list of disjoint,
 * non-empty groups of workers.  SSGD is one group of all workers, ASGD is one
 * group per worker in arrival order (paper Section I); the static x-order mode
 * uses x workers per update and the dynamic x-order mode one worker cluster per
 * update (Section I contribution (2), Section IV-B), clusters taken in
 * ascending order of their slowest member (Section IV-C1, text before Eq. 2).
 * For every element i and every group k in schedule order the library applies
 *
 *     s    = g[m_k0][i] + g[m_k1][i] + ...          members in listed order
 *     gbar = s / |G_k|
 *     d    = fma(wd, p[i], gbar)
 *     v[i] = fma(mu, v[i], d)
 *     p[i] = fma(-lr_k, v[i], p[i])
 *
 * each line one correctly rounded IEEE-754 binary32 operation (bf16 gradients
 * are widened exactly first).  All groups of a round are fused into ONE pass:
 * every scheduled gradient element and p, v are read once, p and v are written
 * once: n * (sum_k |G_k| * sizeof(g) + 16) bytes of traffic per round.
 *
 * A schedule is a CSR pair: group k = group_members[group_offsets[k] ..
 * group_offsets[k+1]).  It need not cover every worker (a round may use only
 * the workers that reported); a worker may appear at most once.
 *
 * Conventions that hold for every entry point
 *   - "device" pointers are CUDA device memory of the current device; "host"
 *     arrays are ordinary memory that is read completely before the call
 *     returns (the caller may free or reuse it at once).
 *   - The caller owns every buffer.  The library allocates no device memory and
 *     keeps no pointer after a call returns, except inside a caller-provided
 *     workspace.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t; NULL = legacy default
 *     stream) and the call returns without synchronizing.  The exceptions are
 *     the calls that copy a table from ordinary host memory (star_multi_prepare,
 *     star_multi_prepare_ex, star_group_update_multi_noalloc): such a copy
 *     makes the host wait until earlier work on `cuda_stream` has finished and
 *     the table is staged, and those calls refuse to run inside a stream
 *     capture (STAR_ERR_UNSUPPORTED, nothing enqueued).
 *   - Every argument error is found on the host BEFORE anything is launched and
 *     leaves p and v untouched.  STAR_ERR_CUDA is a failed launch or runtime
 *     call; star_last_cuda_error() gives its cudaError_t.
 *   - There is no CPU path: without a usable CUDA device the compute entry
 *     points return STAR_ERR_CUDA.
 *   - params, momentum and the scheduled gradient buffers must not overlap.
 *     Element-size alignment is required (4 bytes fp32, 2 bytes bf16).  Buffers
 *     aligned to 32 bytes take the full-width vector path.  So do buffers that
 *     are all views at one common element offset into 32-byte aligned storage
 *     (the usual way a tensor ends up misaligned): up to 7 leading elements are
 *     done one by one and the rest in vectors.  Buffers with no common
 *     alignment phase take a narrower or element-by-element path (slower).
 *     Results are identical on every path.
 */
#ifndef STAR_H_
#define STAR_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define STAR_API __attribute__((visibility("default")))
#else
#define STAR_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    STAR_OK = 0,
    STAR_ERR_NULL_POINTER = 1,      /* a required pointer is NULL */
    STAR_ERR_INVALID_ARG = 2,       /* negative size, bad dtype, misaligned or overlapping buffers */
    STAR_ERR_BAD_SCHEDULE = 3,      /* empty group, duplicate or out-of-range member, bad offsets */
    STAR_ERR_UNSUPPORTED = 4,       /* W above STAR_MAX_WORKERS; a table-copying call inside a stream capture */
    STAR_ERR_WORKSPACE_TOO_SMALL = 5,
    STAR_ERR_CUDA = 6               /* see star_last_cuda_error() */
} star_status_t;

typedef enum { STAR_DTYPE_F32 = 0, STAR_DTYPE_BF16 = 1 } star_dtype_t;

/* Order of the additions inside a group (only rounding depends on it).
 * STAR_SUM_LINEAR: left to right in the listed member order.
 * STAR_SUM_TREE:   pairwise, as gradients are combined along a binary
 *                  aggregation tree (Section IV-D2b: workers add their children's
 *                  gradients to their own on the way up): tree(m_0..m_{c-1}) is the
 *                  member itself for c = 1, else tree(first h) + tree(remaining
 *                  c - h) with h the largest power of two below c. */
typedef enum { STAR_SUM_LINEAR = 0, STAR_SUM_TREE = 1 } star_sum_order_t;

#define STAR_MAX_WORKERS 64

/* Static, NUL-terminated name of a status code. */
STAR_API const char *star_status_string(star_status_t status);

/* cudaError_t of the most recent STAR_ERR_CUDA on the calling thread (0 if none). */
STAR_API int star_last_cuda_error(void);

/* Number of kernels this library has launched in the calling process so far. */
STAR_API int64_t star_launch_count(void);

/* ---------------------------------------------------------------------------
 * Schedule encoding (host only; no CUDA call).  Turns a synchronization-mode
 * decision into the CSR pair.  offsets_out needs room for W + 1 entries,
 * members_out for W entries; *n_groups_out receives K.
 * ------------------------------------------------------------------------- */

/* STAR_OK iff the pair describes n_groups non-empty, pairwise disjoint groups
 * of workers in [0, W) with group_offsets[0] == 0 (Section IV-B: a gradient
 * report feeds exactly one update).  n_groups == 0 is valid. */
STAR_API star_status_t star_schedule_validate(const int32_t *group_offsets, const int32_t *group_members,
                                     int n_groups, int W);

/* Static x-order mode (Section IV-B): consecutive runs of x workers of
 * arrival_order (n_arrived distinct workers, earliest first; NULL = 0..W-1 with
 * n_arrived = W).  x == n_arrived gives SSGD, x == 1 ASGD (Section I).  If x
 * does not divide n_arrived the last group is smaller.  sort_members != 0 lists
 * each group's members in ascending worker index, otherwise in arrival order. */
STAR_API star_status_t star_schedule_static_x(const int32_t *arrival_order, int n_arrived, int W, int x,
                                     int sort_members, int32_t *offsets_out,
                                     int32_t *members_out, int *n_groups_out);

/* Groups from a per-worker label group_of_worker[W] (-1 = worker absent):
 * groups in ascending label order, members in ascending worker index. */
STAR_API star_status_t star_schedule_from_labels(const int32_t *group_of_worker, int W,
                                        int32_t *offsets_out, int32_t *members_out,
                                        int *n_groups_out);

/* Dynamic x-order mode (Section IV-B, ordering of Section IV-C1): one group per
 * cluster id in cluster_of_worker[W] (-1 = absent), groups ascending in the
 * cluster's largest iter_time; ties go to the cluster holding the smaller
 * worker index; members in ascending worker index.  iter_time must be finite. */
STAR_API star_status_t star_schedule_dynamic_x(const double *iter_time, const int32_t *cluster_of_worker,
                                      int W, int32_t *offsets_out, int32_t *members_out,
                                      int *n_groups_out);

/* ---------------------------------------------------------------------------
 * Mode decision (host only): from predicted iteration times to the schedule of
 * the cheapest synchronization mode.  iter_time[w] > 0, finite.
 * ------------------------------------------------------------------------- */

/* Dynamic x-order clustering (Section IV-B): agglomerative hierarchical
 * clustering of the W predicted iteration times with average linkage (mean
 * pairwise |t_a - t_b|).  Merging continues while more than n_clusters clusters
 * remain (n_clusters <= 0: down to one) and the closest pair is no farther
 * apart than max_distance (max_distance < 0: no distance limit).  Equally close
 * pairs: the pair whose clusters hold the smaller worker indices merges first.
 * cluster_of_worker_out[W] receives labels 0..K-1 numbered by each cluster's
 * smallest worker index; *n_clusters_out = K.  Feed the labels to
 * star_schedule_dynamic_x or star_choose_mode. */
STAR_API star_status_t star_cluster_iteration_times(const double *iter_time, int W, int n_clusters,
                                                    double max_distance,
                                                    int32_t *cluster_of_worker_out,
                                                    int *n_clusters_out);

/* Expected time to a fixed training progress per mode (Section IV-C1).
 * T_static_out[x-1], x = 1..W, is Eq. 1: (1 + phi / (x M / W)) * t_x, where t_x,
 * the time one update takes, is read as the x-th smallest iteration time (the
 * moment x gradient reports are in); x = 1 is ASGD, x = W SSGD.  If
 * cluster_of_worker is not NULL (labels >= 0 for every worker), *T_dynamic_out
 * is Eq. 2: 1 / sum_i 1 / ((1 + phi / (n_ci M / W)) * t_ci) over the clusters,
 * n_ci the cluster's size and t_ci its slowest member.  phi is the
 * pre-conditioned gradient noise scale of the current update (>= 0), M the
 * total batch size (> 0); both are the caller's inputs. */
STAR_API star_status_t star_mode_times(const double *iter_time, const int32_t *cluster_of_worker,
                                       int W, double phi, double M, double *T_static_out,
                                       double *T_dynamic_out);

/* The mode with the smallest time and its schedule.  *x_out = x of the chosen
 * static x-order mode, or 0 for the dynamic mode (only if cluster_of_worker is
 * given and Eq. 2 is strictly smaller than every Eq. 1 value); equal static
 * times go to the larger x.  *T_out = that time.  The CSR outputs are as for the
 * schedule encoders: static modes group the workers in ascending predicted time
 * (ties by index) in runs of x, members listed in ascending index; the dynamic
 * mode is star_schedule_dynamic_x on the clusters. */
STAR_API star_status_t star_choose_mode(const double *iter_time, const int32_t *cluster_of_worker,
                                        int W, double phi, double M, int *x_out, double *T_out,
                                        int32_t *offsets_out, int32_t *members_out,
                                        int *n_groups_out);

/* All-reduce architecture (Section IV-B, Section IV-C1 Eq. 3): remove x of the
 * stragglers from the ring, attach each to a parent that waits t_w after the
 * ring's slowest member and adds the gradients of the children that reported
 * by then.  T_a = (1 + phi / ((W - x + q) M / W)) * (t_ring + t_w).
 *   iter_time[w]   predicted iteration time in the ring; a worker is a straggler
 *                  iff (t - min t) / min t > straggler_threshold (Section II: 0.2)
 *   child_time[w]  predicted iteration time of w when attached to a parent; a
 *                  removed worker counts (q) iff child_time[w] - t_ring <= t_w
 *   t_w_max        largest wait considered (t_w in [0, t_w_max])
 * The x slowest stragglers are removed (x = 0..X, at least one worker stays);
 * only t_w = 0 and the waits at which one more child makes it are candidates;
 * ties go to fewer removals, then the shorter wait.  Outputs: *x_out, *t_w_out,
 * *T_out, removed_out[0..x) (slowest first), and the CSR of the ONE group whose
 * gradients enter the update (ring members and children in time, ascending
 * index): on a server holding every worker's buffer the all-reduce mode's
 * update is star_group_update with that schedule. */
STAR_API star_status_t star_choose_all_reduce_mode(const double *iter_time, const double *child_time,
                                                   int W, double phi, double M, double t_w_max,
                                                   double straggler_threshold, int *x_out,
                                                   double *t_w_out, double *T_out,
                                                   int32_t *removed_out, int32_t *offsets_out,
                                                   int32_t *members_out, int *n_groups_out);

/* Parents of the workers taken out of the ring (Section IV-B: each removed
 * straggler reports to a non-straggler with high bandwidth; Section IV-D2a
 * balances the number of children per parent).  Behind a non-blocking switch
 * every ring member is equally near, so the removed workers (removed[0..x), in
 * the order star_choose_all_reduce_mode lists them) are dealt round-robin over
 * the ring members in ascending worker index.  parent_of_out[W] receives the
 * parent of each removed worker and -1 for ring members.  0 <= x < W. */
STAR_API star_status_t star_assign_parents(const int32_t *removed, int x, int W,
                                           int32_t *parent_of_out);

/* Communication tree (Section IV-D2b: the workers of a job form a tree under
 * the parameter server, or under a parent in the all-reduce architecture;
 * workers with longer communication latency sit in lower layers; every worker
 * adds its children's gradients to its own and forwards the sum; the tree is
 * rebuilt before each iteration).  A fanout-ary tree filled layer by layer in
 * ascending latency (ties: the smaller worker index first): the `fanout`
 * quickest workers become children of the root, the next `fanout` children of
 * the quickest worker, and so on.  parent_of_out[W] receives each worker's
 * parent, -1 for the root's children.  latency finite, fanout >= 1. */
STAR_API star_status_t star_build_tree(const double *latency, int W, int fanout, int32_t *parent_of_out);

/* Sharding helper (host only).  The path is elementwise, so a job spread over
 * several parameter servers / GPUs (the paper runs one to N PSs per job,
 * Section III set-up) needs no exchange inside it: rank r of world owns the
 * contiguous element range [*first_out, *first_out + *count_out) of a tensor of
 * n elements.  Ranges are disjoint, cover [0, n), differ in length by less than
 * 2 x `align`, and every range starts at a multiple of `align` elements (use 16 to
 * keep bf16 and fp32 shards on the vector path).  align >= 1. */
STAR_API star_status_t star_shard_range(int64_t n, int world, int rank, int64_t align,
                                        int64_t *first_out, int64_t *count_out);

/* ---------------------------------------------------------------------------
 * Fused grouped update of one flat tensor (the operation defined at the top).
 *   params, momentum : device, fp32, n elements, updated in place
 *   grads            : host array of W device pointers, n elements of
 *                      grad_dtype each; entries of unscheduled workers are
 *                      never dereferenced and may be NULL
 *   group_offsets    : host, n_groups + 1 entries;  group_members : host
 *   lr, mu, wd       : learning rate, momentum coefficient, weight decay
 * n == 0 or n_groups == 0 is a successful no-op.  One kernel launch.
 * ------------------------------------------------------------------------- */
STAR_API star_status_t star_group_update(float *params, float *momentum, const void *const *grads, int W,
                                star_dtype_t grad_dtype, int64_t n,
                                const int32_t *group_offsets, const int32_t *group_members,
                                int n_groups, float lr, float mu, float wd, void *cuda_stream);

/* The same round with one learning rate per group, optional parameter
 * snapshots and a choice of the in-group summation order (sum_order; with
 * groups of more than 4 members the tree order keeps partial sums per element
 * in registers and runs at half the occupancy of the linear order).
 *   lrs        : host, n_groups learning rates.  Section IV-C1 ("Scaling learning
 *                rate after switching") sets the rate of an update built from y
 *                gradient reports to (y / N) x the SSGD rate; the caller computes
 *                the rates, the kernel applies lrs[k] in group k's update.
 *   snapshots  : NULL, or host array of n_groups device pointers (n elements of
 *                snapshot_dtype each, entries may be NULL).  snapshots[k] receives
 *                the parameters as they stand right after group k's update -- the
 *                copy the server sends back to that group's workers (Section II)
 *                -- written in the same pass: fp32 (4 n more bytes of traffic
 *                each) or rounded to bf16, nearest-even (2 n bytes each).
 *                Snapshot buffers must not overlap each other or any other
 *                buffer of the call.
 * Everything else as star_group_update.  One kernel launch. */
STAR_API star_status_t star_group_update_ex(float *params, float *momentum, const void *const *grads,
                                            int W, star_dtype_t grad_dtype, int64_t n,
                                            const int32_t *group_offsets,
                                            const int32_t *group_members, int n_groups,
                                            const float *lrs, float mu, float wd,
                                            void *const *snapshots, star_dtype_t snapshot_dtype,
                                            star_sum_order_t sum_order, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * All-reduce architecture (Section IV-B, paragraph "All-reduce architecture";
 * Section IV-C1, Eq. 3).  Stragglers are taken out of the ring and report their
 * gradients to a parent in the ring; the parent adds the gradients of the
 * children that reported in time to its own, the ring sums its members'
 * aggregates, and one update is made from the gradients of N - x + q workers.
 * Two kernels cover the arithmetic of such a round on one GPU; moving the
 * buffers between GPUs is the caller's (a collective library's) part, and
 * every buffer handed to these calls is memory of the current device.
 * ------------------------------------------------------------------------- */

/* A parent's local aggregate: out[i] = g[m_0][i] + g[m_1][i] + ... over the
 * `count` listed workers (own gradient first, then the children), each addition
 * one binary32 operation, left to right or in tree order (sum_order), written as
 * binary32 (out_dtype F32) or rounded to bf16, nearest even (BF16).
 *   out     : device, n elements of out_dtype; must not overlap a listed buffer
 *   grads   : host array of W device pointers (n elements of grad_dtype each);
 *             only the listed entries are dereferenced
 *   members : host, `count` distinct workers in [0, W); count == 0 is
 *             STAR_ERR_BAD_SCHEDULE (an empty sum has no meaning in this round)
 * n == 0 is a successful no-op.  One kernel launch; n * (count * sizeof(g) +
 * sizeof(out)) bytes of traffic. */
STAR_API star_status_t star_group_reduce(void *out, star_dtype_t out_dtype, const void *const *grads,
                                         int W, star_dtype_t grad_dtype, int64_t n,
                                         const int32_t *members, int count,
                                         star_sum_order_t sum_order, void *cuda_stream);

/* The one update of an all-reduce round from the R ring members' aggregates
 * (binary32, n elements each, device), added left to right in the listed (ring)
 * order; the mean divides by n_reports, the number of gradient reports behind
 * the aggregates (N - x + q of Eq. 3, R <= n_reports <= 255):
 *     s = sums[0][i] + sums[1][i] + ... ; gbar = s / n_reports ;
 *     d = fma(wd, p, gbar) ; v = fma(mu, v, d) ; p = fma(-lr, v, p)
 * sums: host array of R device pointers.  Every rank that applies this call to
 * the same aggregates in the same order holds bit-identical parameters
 * afterwards.  R == 0 with n_reports == 0, or n == 0, is a no-op.  One launch. */
STAR_API star_status_t star_group_update_from_sums(float *params, float *momentum,
                                                   const float *const *sums, int R, int64_t n,
                                                   int n_reports, float lr, float mu, float wd,
                                                   void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Fused grouped update of a LIST of tensors (per-layer parameters) in one
 * launch.  The pointer table and tile map live in a caller-provided device
 * workspace that is prepared once per tensor list and reused every round.
 * ------------------------------------------------------------------------- */

/* Host-side description of a prepared tensor list.  Plain data, filled by
 * star_multi_prepare and passed back by value-pointer every round; it holds
 * the workspace address but owns nothing. */
typedef struct {
    uint64_t magic;            /* set by star_multi_prepare; anything else is rejected */
    const void *d_workspace;   /* the caller's device workspace */
    int64_t total_elements;    /* sum of the tensor sizes */
    int64_t n_tiles;           /* work items the kernel walks */
    uint64_t complete_workers; /* bit w set: worker w has a gradient for every non-empty tensor */
    int32_t n_tensors;
    int32_t W;
    int32_t grad_dtype;        /* star_dtype_t */
    int32_t tile_elements;     /* elements per tile */
    int32_t n_snapshot_sets;   /* snapshot buffer sets registered by star_multi_prepare_ex (else 0) */
    int32_t snapshot_dtype;    /* star_dtype_t of those buffers */
} star_multi_plan_t;

/* Bytes of device workspace needed for n_tensors tensors of the given sizes
 * (host array, elements per tensor, 0 allowed) and W workers (no snapshot sets). */
STAR_API star_status_t star_multi_workspace_bytes(int n_tensors, const int64_t *sizes, int W,
                                         size_t *bytes_out);

/* Fill the workspace and *plan_out.  params, momentum: host arrays of n_tensors
 * device pointers; grads: host array of n_tensors * W device pointers, entry
 * [t * W + w] = worker w's gradient for tensor t (NULL allowed for workers that
 * will never be scheduled); sizes: host, elements per tensor.  d_workspace:
 * device, 256-byte aligned, at least star_multi_workspace_bytes() bytes.  The
 * table is built in ordinary host memory and copied with one cudaMemcpyAsync on
 * cuda_stream; the host copy is released before the call returns (a copy from
 * pageable memory returns once the data is staged, which makes the host wait
 * for earlier work on cuda_stream), later work on the same stream sees the
 * table.  Inside a stream capture the call returns STAR_ERR_UNSUPPORTED and
 * enqueues nothing.  No buffer that a round writes (params, momentum) may
 * share memory with any other buffer of the list, in the same or in another
 * tensor (STAR_ERR_INVALID_ARG: e.g. a tied weight listed twice); gradient
 * buffers may alias one another.  Not a per-round call: once per tensor list. */
STAR_API star_status_t star_multi_prepare(int n_tensors, float *const *params, float *const *momentum,
                                 const void *const *grads, const int64_t *sizes, int W,
                                 star_dtype_t grad_dtype, void *d_workspace,
                                 size_t workspace_bytes, void *cuda_stream,
                                 star_multi_plan_t *plan_out);

/* One round over the prepared list: the same operation as star_group_update on
 * every tensor, one kernel launch in total.  Scheduling a worker whose gradient
 * pointer was NULL for some non-empty tensor at prepare time is rejected with
 * STAR_ERR_NULL_POINTER.  A plan not made by star_multi_prepare is rejected
 * with STAR_ERR_INVALID_ARG. */
STAR_API star_status_t star_group_update_multi(const star_multi_plan_t *plan,
                                      const int32_t *group_offsets, const int32_t *group_members,
                                      int n_groups, float lr, float mu, float wd,
                                      void *cuda_stream);

/* The tensor-list round with one learning rate per group (lrs: host, n_groups
 * values; Section IV-C1 rate scaling).  Otherwise as star_group_update_multi. */
STAR_API star_status_t star_group_update_multi_lrs(const star_multi_plan_t *plan,
                                                   const int32_t *group_offsets,
                                                   const int32_t *group_members, int n_groups,
                                                   const float *lrs, float mu, float wd,
                                                   void *cuda_stream);

/* Tensor lists with parameter snapshots and the tree order.  A snapshot SET is
 * one buffer per tensor of the list; up to STAR_MAX_WORKERS sets are registered
 * when the list is prepared (their pointers go into the same workspace table),
 * and every round says which set, if any, receives the parameters as they stand
 * right after each group's update -- the copy the server sends back to that
 * group's workers (Section II) -- written in the same pass.
 *   star_multi_workspace_bytes_ex : workspace size with n_snapshot_sets sets
 *   star_multi_prepare_ex         : as star_multi_prepare, plus
 *       snapshots      host array of n_tensors * n_snapshot_sets device pointers,
 *                      entry [t * n_snapshot_sets + s] = tensor t's buffer of set
 *                      s (sizes[t] elements of snapshot_dtype; NULL = tensor t is
 *                      not captured by set s); snapshot buffers are written, so
 *                      they must not overlap anything else in the list
 *   star_group_update_multi_ex    : one round, one launch, with
 *       lrs                    host, one learning rate per group (Section IV-C1)
 *       snapshot_set_of_group  NULL, or host array of n_groups entries: the set
 *                              (0 .. n_snapshot_sets-1) written after group k, or -1
 *       sum_order              STAR_SUM_LINEAR or STAR_SUM_TREE (Section IV-D2b)
 * Results equal star_group_update_ex applied to every tensor of the list. */
STAR_API star_status_t star_multi_workspace_bytes_ex(int n_tensors, const int64_t *sizes, int W,
                                                     int n_snapshot_sets, size_t *bytes_out);

STAR_API star_status_t star_multi_prepare_ex(int n_tensors, float *const *params, float *const *momentum,
                                             const void *const *grads, const int64_t *sizes, int W,
                                             star_dtype_t grad_dtype, int n_snapshot_sets,
                                             void *const *snapshots, star_dtype_t snapshot_dtype,
                                             void *d_workspace, size_t workspace_bytes,
                                             void *cuda_stream, star_multi_plan_t *plan_out);

STAR_API star_status_t star_group_update_multi_ex(const star_multi_plan_t *plan,
                                                  const int32_t *group_offsets,
                                                  const int32_t *group_members, int n_groups,
                                                  const float *lrs, float mu, float wd,
                                                  const int32_t *snapshot_set_of_group,
                                                  star_sum_order_t sum_order, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Fused grouped update with the state and the gradients in HOST memory (the
 * paper's parameter server keeps its parameter and gradient copies in host
 * memory, Section II).  Same operation and results as star_group_update; the
 * data is streamed through the GPU in chunks: copy a chunk of p, v and of every
 * scheduled worker's gradient to the device, run the fused kernel on it, copy
 * p and v back, with the copies of neighbouring chunks overlapping (host to
 * device on cuda_stream, device to host on an internal stream).
 *   h_params, h_momentum : host, fp32, n elements, updated in place
 *   h_grads              : host array of W host pointers (unscheduled: may be NULL)
 *   d_workspace          : device, 256-byte aligned staging memory provided by
 *                          the caller; star_host_workspace_bytes() gives the
 *                          size for a chosen chunk length
 * Host buffers should be page-locked (cudaHostAlloc / cudaHostRegister):
 * pageable memory works but its copies do not overlap.  The call enqueues all
 * work and returns; results are in the host buffers once cuda_stream has been
 * synchronized.  The first call on a device creates one internal stream and a
 * few events (no device memory).  Calls on the same device are serialized
 * against each other at enqueue time by the library; they must not share a
 * workspace unless they are ordered on one stream.
 * ------------------------------------------------------------------------- */

/* Workspace bytes for chunks of chunk_elements elements (a multiple of 2048, at
 * least 2048) when at most max_scheduled workers are scheduled in a round. */
STAR_API star_status_t star_host_workspace_bytes(int max_scheduled, star_dtype_t grad_dtype,
                                                 int64_t chunk_elements, size_t *bytes_out);

/* The chunk length is the largest multiple of 2048 that fits workspace_bytes for
 * the number of workers this schedule uses; STAR_ERR_WORKSPACE_TOO_SMALL if
 * that is below 2048.  One kernel launch per chunk. */
STAR_API star_status_t star_group_update_host(float *h_params, float *h_momentum,
                                              const void *const *h_grads, int W,
                                              star_dtype_t grad_dtype, int64_t n,
                                              const int32_t *group_offsets,
                                              const int32_t *group_members, int n_groups, float lr,
                                              float mu, float wd, void *d_workspace,
                                              size_t workspace_bytes, void *cuda_stream);

/* The host-buffer round with one learning rate per group (lrs: host, n_groups
 * values; Section IV-C1), optional parameter snapshots into HOST buffers
 * (h_snapshots: NULL, or host array of n_groups host pointers, n elements of
 * snapshot_dtype each, entries may be NULL: the copy of the parameters after
 * that group's update that the server sends back to the group's workers,
 * Section II) and the choice of summation order.  Snapshot chunks are staged in
 * the workspace and copied back with p and v; star_host_workspace_bytes_ex sizes
 * the workspace for up to max_snapshots snapshots of snapshot_dtype per round.
 * Everything else as star_group_update_host. */
STAR_API star_status_t star_host_workspace_bytes_ex(int max_scheduled, star_dtype_t grad_dtype,
                                                    int max_snapshots, star_dtype_t snapshot_dtype,
                                                    int64_t chunk_elements, size_t *bytes_out);

STAR_API star_status_t star_group_update_host_ex(float *h_params, float *h_momentum,
                                                 const void *const *h_grads, int W,
                                                 star_dtype_t grad_dtype, int64_t n,
                                                 const int32_t *group_offsets,
                                                 const int32_t *group_members, int n_groups,
                                                 const float *lrs, float mu, float wd,
                                                 void *const *h_snapshots, star_dtype_t snapshot_dtype,
                                                 star_sum_order_t sum_order, void *d_workspace,
                                                 size_t workspace_bytes, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Tensor-list round for callers that cannot allocate device memory.
 *
 * The paper has no counterpart to this entry point; it exists for integration.
 * Some callers of this library are not in a position to call cudaMalloc or to
 * obtain a workspace from an allocator: a plug-in that runs inside another
 * framework's step after that framework's pool has taken all free device
 * memory, a hook on a latency-critical path where cudaMalloc's device-wide
 * synchronization is not acceptable, or early start-up code that runs before
 * any allocator exists.  For them the pointer table and tile map that
 * star_multi_prepare would place in a caller workspace live in a fixed array of
 * STAR_STATIC_SCRATCH_BYTES inside the library's device image (each GPU that
 * loads the library holds that much until the process exits).
 *
 * The call does the work of star_multi_prepare followed by
 * star_group_update_multi: arguments have the same meaning as there, and the
 * results are identical.  It calls no cudaMalloc, cudaFree or other allocating
 * routine.  Differences to know about:
 *   - Size limit: a list whose table needs more than STAR_STATIC_SCRATCH_BYTES
 *     (see star_multi_workspace_bytes) is rejected with
 *     STAR_ERR_WORKSPACE_TOO_SMALL and nothing is launched.  1 MiB covers, for
 *     example, 292 tensors / 355 M elements / 16 workers (about 0.75 MiB).
 *   - The first call on each device looks up the array's device address (with
 *     that device current).
 *   - The call cannot be part of a stream capture, first call or not: the table
 *     is copied from host memory that is released on return, which a captured
 *     graph would read again at every replay.  When cuda_stream is capturing
 *     the call returns STAR_ERR_UNSUPPORTED and enqueues nothing.
 *   - All calls on a device share the one array, and it keeps the previous
 *     call's table; each call rewrites the part it uses before its kernel
 *     reads it, so nothing has to start out zeroed.  Calls on one stream are
 *     ordered and safe.  Calls that can overlap on the GPU (different streams
 *     without a dependency, or several host threads) race on the array: the
 *     caller must serialize them.
 *   - The table is rebuilt and copied (one cudaMemcpyAsync from pageable host
 *     memory) on every call.  That copy makes the host wait until the work
 *     queued earlier on cuda_stream, the previous round included, has finished:
 *     the call does not run ahead of the GPU.  Callers that can provide a
 *     workspace should prepare once and use star_group_update_multi.
 * ------------------------------------------------------------------------- */
#define STAR_STATIC_SCRATCH_BYTES (1u << 20)

STAR_API star_status_t star_group_update_multi_noalloc(
    int n_tensors, float *const *params, float *const *momentum, const void *const *grads,
    const int64_t *sizes, int W, star_dtype_t grad_dtype, const int32_t *group_offsets,
    const int32_t *group_members, int n_groups, float lr, float mu, float wd, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* STAR_H_ */
