// C-ABI entry points: argument checks on the host, then one kernel launch.
#include <algorithm>
#include <atomic>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <vector>

#include <cuda_runtime.h>

#include "kernels.cuh"
#include "star.h"

namespace {

using namespace star;

thread_local int g_last_cuda_error = 0;
std::atomic<int64_t> g_launches{0};

star_status_t cuda_failed(cudaError_t e)
{
    g_last_cuda_error = static_cast<int>(e);
    return STAR_ERR_CUDA;
}

constexpr uint64_t kPlanMagic = 0x53544152504c414eull;   // "STARPLAN"
constexpr size_t kWorkspaceAlign = 256;

// ---------------------------------------------------------------------------
// Launch geometry: a persistent grid of (SM count x resident blocks) blocks,
// capped by the work there is.  Queried once per device and kernel.
// ---------------------------------------------------------------------------
constexpr int kMaxDevices = 64;

struct Geometry {
    std::atomic<int> blocks{0};
};

template <typename Kernel>
cudaError_t resident_blocks(Kernel kernel, Geometry *cache, int *blocks_out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    int blocks = cache[dev].blocks.load(std::memory_order_relaxed);
    if (blocks == 0) {
        int sms = 0, per_sm = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kBlockThreads, 0);
        if (e != cudaSuccess) return e;
        if (per_sm < 1) per_sm = 1;
        blocks = sms * per_sm;
        cache[dev].blocks.store(blocks, std::memory_order_relaxed);
    }
    *blocks_out = blocks;
    return cudaSuccess;
}

// Grid for `work` blocks' worth of tiles when `resident` blocks fit on the
// device at once.  Up to kPersistentWaves waves of work run as a persistent
// grid (every block strides over the tiles); beyond that one block per tile.
// Measured on B200: the persistent grid is ~3 % faster at 21 waves
// (ResNet-50-sized), one block per tile ~1-3 % faster at 114 and 280 waves
// (VGG-16- and BERT-large-sized).  Both kernels loop with a grid stride, so
// either choice is correct for any size.
constexpr int64_t kPersistentWaves = 32;

int choose_grid(int64_t work, int resident)
{
    if (work < 1) return 1;
    if (work <= resident) return static_cast<int>(work);
    if (work <= kPersistentWaves * resident) return resident;
    return static_cast<int>(work < 0x7fffffff ? work : 0x7fffffff);
}

// ---------------------------------------------------------------------------
// Schedule: validate, then flatten into the kernel's slot list.  lrs (one rate
// per group) overrides the single rate lr when given.
// ---------------------------------------------------------------------------
star_status_t flatten_schedule(const int32_t *group_offsets, const int32_t *group_members, int n_groups,
                               int W, float lr, FlatSchedule *out, const float *lrs)
{
    const star_status_t st = star_schedule_validate(group_offsets, group_members, n_groups, W);
    if (st != STAR_OK) return st;
    std::memset(out, 0, sizeof *out);
    out->n_slots = n_groups > 0 ? group_offsets[n_groups] : 0;
    for (int k = 0; k < n_groups; ++k) {
        const int first = group_offsets[k], last = group_offsets[k + 1];
        for (int j = first; j < last; ++j) {
            out->member[j] = static_cast<uint8_t>(group_members[j]);
        }
        out->size_at_start[first] = static_cast<uint8_t>(last - first);
        out->group_size[last - 1] = static_cast<uint8_t>(last - first);
        out->neg_lr[last - 1] = lrs ? -lrs[k] : -lr;
    }
    return STAR_OK;
}

bool overlaps(const void *a, size_t a_bytes, const void *b, size_t b_bytes)
{
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + b_bytes && b0 < a0 + a_bytes;
}

bool aligned(const void *p, size_t bytes) { return reinterpret_cast<uintptr_t>(p) % bytes == 0; }

// Kernel choices.  bf16: 8 elements per thread (one 16-byte gradient load per
// worker, 32 bytes each of p and v); fp32: 4 elements per thread; 4 gradient
// loads in flight per thread.
constexpr int kVecBF16 = 8;
constexpr int kVecF32 = 4;
constexpr int kDepthVector = 4;
constexpr int kDepthNarrow = 8;           // flat kernels whose gradient loads are narrower than 16 bytes
constexpr int kVecBF16Half = 4;           // bf16 with buffers aligned for 16-byte state / 8-byte gradient accesses

// The device buffers one thread's vector touches (of a call, or of one tensor
// of a list), with their element sizes.
struct Buffers {
    struct Item {
        uintptr_t addr;
        unsigned elem;
    };
    Item item[2 + 2 * kMaxWorkers];
    int count = 0;
    void add(const void *p, unsigned elem) { item[count++] = Item{reinterpret_cast<uintptr_t>(p), elem}; }
};

// Elements per thread and the number of leading elements in front of the
// vector body.  A vector of `vec` elements needs every buffer aligned to vec
// elements of its own type (bf16, vec 8: 32 bytes for fp32 state, 16 bytes for
// gradients) at the element where the body starts.  Buffers that are views at
// one common element offset into aligned storage reach that alignment together
// after `head` < vec elements, which are then done one by one; buffers with no
// common phase fall back to a narrower vector (bf16 flat kernels: 4) or to the
// element-by-element kernel (vec 1).  Results do not depend on the choice.
struct VectorPlan {
    int vec = 1;
    int head = 0;
};

VectorPlan plan_vector(star_dtype_t dt, const Buffers &b, int64_t n, bool allow_half)
{
    const int candidates[2] = {dt == STAR_DTYPE_BF16 ? kVecBF16 : kVecF32,
                               dt == STAR_DTYPE_BF16 && allow_half ? kVecBF16Half : 0};
    for (int vec : candidates) {
        if (vec <= 1 || b.count == 0) continue;
        const Buffers::Item &f = b.item[0];
        const unsigned span = f.elem * static_cast<unsigned>(vec);
        const unsigned r = static_cast<unsigned>(f.addr % span);
        const int head = r == 0 ? 0 : static_cast<int>((span - r) / f.elem);
        bool ok = true;
        for (int i = 0; i < b.count && ok; ++i) {
            const Buffers::Item &x = b.item[i];
            ok = (x.addr + static_cast<uintptr_t>(head) * x.elem) % (x.elem * static_cast<unsigned>(vec)) == 0;
        }
        if (ok && n >= head + vec) return VectorPlan{vec, head};
    }
    return VectorPlan{};
}

// Launch of a grid-stride kernel over n_vec vectors of one flat tensor.
template <typename Kernel, typename Args>
star_status_t launch_grid_stride(Kernel kernel, Geometry *cache, const Args &args, int64_t n_vec, cudaStream_t stream)
{
    int blocks = 0;
    cudaError_t e = resident_blocks(kernel, cache, &blocks);
    if (e != cudaSuccess) return cuda_failed(e);
    const int64_t work = (n_vec + kBlockThreads - 1) / kBlockThreads;
    const int grid = choose_grid(work, blocks);
    kernel<<<grid, kBlockThreads, 0, stream>>>(args);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_failed(e);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return STAR_OK;
}

template <typename G, int VEC>
star_status_t launch_flat(const FlatArgs &args, cudaStream_t stream)
{
    static Geometry cache[kMaxDevices];
    // Narrow loads (element by element, half-width bf16) keep more of them in flight.
    constexpr int depth = VEC * G::kBytes >= 16 ? kDepthVector : kDepthNarrow;
    return launch_grid_stride(star_update_flat_kernel<G, VEC, depth>, cache, args, (args.n - args.head) / VEC, stream);
}

}  // namespace

extern "C" const char *star_status_string(star_status_t status)
{
    switch (status) {
    case STAR_OK: return "STAR_OK";
    case STAR_ERR_NULL_POINTER: return "STAR_ERR_NULL_POINTER";
    case STAR_ERR_INVALID_ARG: return "STAR_ERR_INVALID_ARG";
    case STAR_ERR_BAD_SCHEDULE: return "STAR_ERR_BAD_SCHEDULE";
    case STAR_ERR_UNSUPPORTED: return "STAR_ERR_UNSUPPORTED";
    case STAR_ERR_WORKSPACE_TOO_SMALL: return "STAR_ERR_WORKSPACE_TOO_SMALL";
    case STAR_ERR_CUDA: return "STAR_ERR_CUDA";
    }
    return "STAR_ERR_UNKNOWN";
}

extern "C" int star_last_cuda_error(void) { return g_last_cuda_error; }

extern "C" int64_t star_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

namespace {

// Everything the flat entry points check before a launch.  On STAR_OK either
// *noop is set (empty tensor or empty schedule: nothing to do) or *args is
// complete (but for args->head) and *buffers lists the buffers of the call.
star_status_t prepare_flat(float *params, float *momentum, const void *const *grads, int W,
                           star_dtype_t grad_dtype, int64_t n, const int32_t *group_offsets,
                           const int32_t *group_members, int n_groups, float lr, const float *lrs, float mu,
                           float wd, FlatArgs *args, Buffers *buffers, bool *noop)
{
    *noop = false;
    if (n < 0 || W < 0) return STAR_ERR_INVALID_ARG;
    if (grad_dtype != STAR_DTYPE_F32 && grad_dtype != STAR_DTYPE_BF16) return STAR_ERR_INVALID_ARG;
    if (W > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    const star_status_t st = flatten_schedule(group_offsets, group_members, n_groups, W, lr, &args->sched, lrs);
    if (st != STAR_OK) return st;
    if (n == 0 || n_groups == 0) {
        *noop = true;
        return STAR_OK;
    }
    if (!params || !momentum || !grads) return STAR_ERR_NULL_POINTER;
    const unsigned gsize = grad_dtype == STAR_DTYPE_BF16 ? 2 : 4;
    const size_t state_bytes = static_cast<size_t>(n) * 4, grad_bytes = static_cast<size_t>(n) * gsize;
    if (!aligned(params, 4) || !aligned(momentum, 4)) return STAR_ERR_INVALID_ARG;
    if (overlaps(params, state_bytes, momentum, state_bytes)) return STAR_ERR_INVALID_ARG;
    buffers->add(params, 4);
    buffers->add(momentum, 4);
    std::memset(args->grads, 0, sizeof args->grads);
    for (int j = 0; j < args->sched.n_slots; ++j) {
        const int w = args->sched.member[j];
        const void *g = grads[w];
        if (!g) return STAR_ERR_NULL_POINTER;
        if (!aligned(g, gsize)) return STAR_ERR_INVALID_ARG;
        if (overlaps(g, grad_bytes, params, state_bytes) || overlaps(g, grad_bytes, momentum, state_bytes))
            return STAR_ERR_INVALID_ARG;
        buffers->add(g, gsize);
        args->grads[w] = g;
    }
    args->params = params;
    args->momentum = momentum;
    args->n = n;
    args->head = 0;
    args->hyper = Hyper{mu, wd};
    return STAR_OK;
}

star_status_t dispatch_flat(FlatArgs &args, star_dtype_t grad_dtype, const VectorPlan &plan, cudaStream_t stream)
{
    args.head = plan.head;
    if (grad_dtype == STAR_DTYPE_BF16) {
        if (plan.vec == kVecBF16) return launch_flat<GradBF16, kVecBF16>(args, stream);
        if (plan.vec == kVecBF16Half) return launch_flat<GradBF16, kVecBF16Half>(args, stream);
        return launch_flat<GradBF16, 1>(args, stream);
    }
    return plan.vec == kVecF32 ? launch_flat<GradF32, kVecF32>(args, stream) : launch_flat<GradF32, 1>(args, stream);
}

template <typename G, int VEC, int TREE>
star_status_t launch_flat_snapshot(const SnapshotArgs &args, cudaStream_t stream)
{
    static Geometry cache[kMaxDevices];
    return launch_grid_stride(star_update_flat_snapshot_kernel<G, VEC, kDepthVector, TREE>, cache, args,
                              (args.flat.n - args.flat.head) / VEC, stream);
}

// The extended kernels come in the full vector width and element by element only.
template <typename G, int VEC, int TREE>
star_status_t dispatch_snapshot(SnapshotArgs &args, const VectorPlan &plan, cudaStream_t stream)
{
    args.flat.head = plan.head;
    return plan.vec == VEC ? launch_flat_snapshot<G, VEC, TREE>(args, stream)
                           : launch_flat_snapshot<G, 1, TREE>(args, stream);
}

// Span of the tree-order kernel that serves groups of up to `largest` members
// (0: the linear kernel; up to two members both orders are the same sum).
int tree_span(star_sum_order_t order, int largest)
{
    if (order != STAR_SUM_TREE || largest <= 2) return 0;
    return largest <= 4 ? 4 : largest <= 16 ? 16 : 64;
}

int largest_group(const int32_t *group_offsets, int n_groups)
{
    int largest = 1;
    for (int k = 0; k < n_groups; ++k) largest = std::max(largest, group_offsets[k + 1] - group_offsets[k]);
    return largest;
}

// The snapshot / tree-order kernel for a tree span (0: linear order).
star_status_t dispatch_extended(SnapshotArgs &sargs, star_dtype_t grad_dtype, const VectorPlan &plan, int tree,
                                cudaStream_t stream)
{
    const bool bf16 = grad_dtype == STAR_DTYPE_BF16;
    switch (tree) {
    case 4: return bf16 ? dispatch_snapshot<GradBF16, kVecBF16, 4>(sargs, plan, stream)
                        : dispatch_snapshot<GradF32, kVecF32, 4>(sargs, plan, stream);
    case 16: return bf16 ? dispatch_snapshot<GradBF16, kVecBF16, 16>(sargs, plan, stream)
                         : dispatch_snapshot<GradF32, kVecF32, 16>(sargs, plan, stream);
    case 64: return bf16 ? dispatch_snapshot<GradBF16, kVecBF16, 64>(sargs, plan, stream)
                         : dispatch_snapshot<GradF32, kVecF32, 64>(sargs, plan, stream);
    default: return bf16 ? dispatch_snapshot<GradBF16, kVecBF16, 0>(sargs, plan, stream)
                         : dispatch_snapshot<GradF32, kVecF32, 0>(sargs, plan, stream);
    }
}

}  // namespace

extern "C" star_status_t star_group_update(float *params, float *momentum, const void *const *grads, int W,
                                           star_dtype_t grad_dtype, int64_t n,
                                           const int32_t *group_offsets, const int32_t *group_members,
                                           int n_groups, float lr, float mu, float wd, void *cuda_stream)
{
    FlatArgs args;
    Buffers buffers;
    bool noop = false;
    const star_status_t st = prepare_flat(params, momentum, grads, W, grad_dtype, n, group_offsets, group_members,
                                          n_groups, lr, nullptr, mu, wd, &args, &buffers, &noop);
    if (st != STAR_OK || noop) return st;
    return dispatch_flat(args, grad_dtype, plan_vector(grad_dtype, buffers, n, true),
                         static_cast<cudaStream_t>(cuda_stream));
}

// Per-group learning rates and parameter snapshots.
extern "C" star_status_t star_group_update_ex(float *params, float *momentum, const void *const *grads,
                                              int W, star_dtype_t grad_dtype, int64_t n,
                                              const int32_t *group_offsets, const int32_t *group_members,
                                              int n_groups, const float *lrs, float mu, float wd,
                                              void *const *snapshots, star_dtype_t snapshot_dtype,
                                              star_sum_order_t sum_order, void *cuda_stream)
{
    if (sum_order != STAR_SUM_LINEAR && sum_order != STAR_SUM_TREE) return STAR_ERR_INVALID_ARG;
    if (snapshot_dtype != STAR_DTYPE_F32 && snapshot_dtype != STAR_DTYPE_BF16) return STAR_ERR_INVALID_ARG;
    if (n_groups > 0 && !lrs) return STAR_ERR_NULL_POINTER;
    SnapshotArgs sargs;
    FlatArgs &args = sargs.flat;
    Buffers buffers;
    bool noop = false;
    const star_status_t st = prepare_flat(params, momentum, grads, W, grad_dtype, n, group_offsets, group_members,
                                          n_groups, 0.0f, lrs, mu, wd, &args, &buffers, &noop);
    if (st != STAR_OK || noop) return st;

    const size_t gsize = grad_dtype == STAR_DTYPE_BF16 ? 2 : 4;
    const size_t state_bytes = static_cast<size_t>(n) * 4, grad_bytes = static_cast<size_t>(n) * gsize;
    std::memset(sargs.snapshots, 0, sizeof sargs.snapshots);
    sargs.snapshot_bf16 = snapshot_dtype == STAR_DTYPE_BF16 ? 1 : 0;
    const unsigned snap_elem = snapshot_dtype == STAR_DTYPE_BF16 ? 2 : 4;
    const size_t snap_bytes = static_cast<size_t>(n) * snap_elem;
    bool any_snapshot = false;
    for (int k = 0; snapshots && k < n_groups; ++k) {
        void *snap = snapshots[k];
        if (!snap) continue;
        if (!aligned(snap, snap_elem)) return STAR_ERR_INVALID_ARG;
        if (overlaps(snap, snap_bytes, params, state_bytes) || overlaps(snap, snap_bytes, momentum, state_bytes))
            return STAR_ERR_INVALID_ARG;
        for (int j = 0; j < args.sched.n_slots; ++j)
            if (overlaps(snap, snap_bytes, args.grads[args.sched.member[j]], grad_bytes)) return STAR_ERR_INVALID_ARG;
        for (int l = 0; l < k; ++l)
            if (snapshots[l] && overlaps(snap, snap_bytes, snapshots[l], snap_bytes)) return STAR_ERR_INVALID_ARG;
        buffers.add(snap, snap_elem);
        sargs.snapshots[group_offsets[k + 1] - 1] = snap;
        any_snapshot = true;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int tree = tree_span(sum_order, largest_group(group_offsets, n_groups));
    if (tree == 0 && !any_snapshot)        // per-group rates only
        return dispatch_flat(args, grad_dtype, plan_vector(grad_dtype, buffers, n, true), stream);
    return dispatch_extended(sargs, grad_dtype, plan_vector(grad_dtype, buffers, n, false), tree, stream);
}

// ---------------------------------------------------------------------------
// All-reduce architecture: a parent's local sum, and the update from the ring
// members' sums.
// ---------------------------------------------------------------------------
namespace {

template <typename G, int VEC, int TREE>
star_status_t launch_reduce(const ReduceArgs &args, cudaStream_t stream)
{
    static Geometry cache[kMaxDevices];
    constexpr int depth = VEC * G::kBytes >= 16 ? kDepthVector : kDepthNarrow;
    return launch_grid_stride(star_group_reduce_kernel<G, VEC, depth, TREE>, cache, args,
                              (args.n - args.head) / VEC, stream);
}

template <typename G, int VEC>
star_status_t dispatch_reduce(ReduceArgs &args, const VectorPlan &plan, int tree, cudaStream_t stream)
{
    args.head = plan.head;
    const bool vec = plan.vec == VEC;
    if (vec && args.count <= 2) {          // too few loads per vector: two vectors per thread
        static Geometry cache[kMaxDevices];
        return launch_grid_stride(star_group_reduce_pair_kernel<G, VEC>, cache, args, (args.n - args.head) / VEC / 2,
                                  stream);
    }
    switch (tree) {
    case 4: return vec ? launch_reduce<G, VEC, 4>(args, stream) : launch_reduce<G, 1, 4>(args, stream);
    case 16: return vec ? launch_reduce<G, VEC, 16>(args, stream) : launch_reduce<G, 1, 16>(args, stream);
    case 64: return vec ? launch_reduce<G, VEC, 64>(args, stream) : launch_reduce<G, 1, 64>(args, stream);
    default: return vec ? launch_reduce<G, VEC, 0>(args, stream) : launch_reduce<G, 1, 0>(args, stream);
    }
}

}  // namespace

extern "C" star_status_t star_group_reduce(void *out, star_dtype_t out_dtype, const void *const *grads, int W,
                                           star_dtype_t grad_dtype, int64_t n, const int32_t *members,
                                           int count, star_sum_order_t sum_order, void *cuda_stream)
{
    if (n < 0 || W < 0 || count < 0) return STAR_ERR_INVALID_ARG;
    if (grad_dtype != STAR_DTYPE_F32 && grad_dtype != STAR_DTYPE_BF16) return STAR_ERR_INVALID_ARG;
    if (out_dtype != STAR_DTYPE_F32 && out_dtype != STAR_DTYPE_BF16) return STAR_ERR_INVALID_ARG;
    if (sum_order != STAR_SUM_LINEAR && sum_order != STAR_SUM_TREE) return STAR_ERR_INVALID_ARG;
    if (W > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    if (count == 0) return STAR_ERR_BAD_SCHEDULE;           // the sum of nothing is not defined here
    if (!members) return STAR_ERR_NULL_POINTER;
    const int32_t one_group[2] = {0, count};
    const star_status_t st = star_schedule_validate(one_group, members, 1, W);
    if (st != STAR_OK) return st;
    if (n == 0) return STAR_OK;
    if (!out || !grads) return STAR_ERR_NULL_POINTER;

    const unsigned gsize = grad_dtype == STAR_DTYPE_BF16 ? 2 : 4, osize = out_dtype == STAR_DTYPE_BF16 ? 2 : 4;
    const size_t grad_bytes = static_cast<size_t>(n) * gsize, out_bytes = static_cast<size_t>(n) * osize;
    if (!aligned(out, osize)) return STAR_ERR_INVALID_ARG;
    ReduceArgs args;
    std::memset(&args, 0, sizeof args);
    Buffers buffers;
    buffers.add(out, osize);
    for (int j = 0; j < count; ++j) {
        const void *g = grads[members[j]];
        if (!g) return STAR_ERR_NULL_POINTER;
        if (!aligned(g, gsize)) return STAR_ERR_INVALID_ARG;
        if (overlaps(g, grad_bytes, out, out_bytes)) return STAR_ERR_INVALID_ARG;
        buffers.add(g, gsize);
        args.src[j] = g;
    }
    args.out = out;
    args.n = n;
    args.count = count;
    args.out_bf16 = out_dtype == STAR_DTYPE_BF16 ? 1 : 0;
    const VectorPlan plan = plan_vector(grad_dtype, buffers, n, false);
    const int tree = tree_span(sum_order, count);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    return grad_dtype == STAR_DTYPE_BF16 ? dispatch_reduce<GradBF16, kVecBF16>(args, plan, tree, stream)
                                         : dispatch_reduce<GradF32, kVecF32>(args, plan, tree, stream);
}

extern "C" star_status_t star_group_update_from_sums(float *params, float *momentum, const float *const *sums,
                                                     int R, int64_t n, int n_reports, float lr, float mu,
                                                     float wd, void *cuda_stream)
{
    if (R < 0 || n < 0) return STAR_ERR_INVALID_ARG;
    if (R > STAR_MAX_WORKERS || n_reports > 255) return STAR_ERR_UNSUPPORTED;
    if (R == 0) return n_reports == 0 ? STAR_OK : STAR_ERR_INVALID_ARG;
    if (n_reports < R) return STAR_ERR_INVALID_ARG;
    int32_t members[STAR_MAX_WORKERS];
    for (int r = 0; r < R; ++r) members[r] = r;
    const int32_t one_group[2] = {0, R};
    FlatArgs args;
    Buffers buffers;
    bool noop = false;
    const star_status_t st =
        prepare_flat(params, momentum, reinterpret_cast<const void *const *>(sums), R, STAR_DTYPE_F32, n, one_group,
                     members, 1, lr, nullptr, mu, wd, &args, &buffers, &noop);
    if (st != STAR_OK || noop) return st;
    // The mean is taken over the gradient reports behind the sums, not over the sums.
    args.sched.group_size[R - 1] = static_cast<uint8_t>(n_reports);
    return dispatch_flat(args, STAR_DTYPE_F32, plan_vector(STAR_DTYPE_F32, buffers, n, false),
                         static_cast<cudaStream_t>(cuda_stream));
}

// ---------------------------------------------------------------------------
// Tensor lists.
// ---------------------------------------------------------------------------
namespace {

constexpr int64_t tile_elements(star_dtype_t dt)
{
    return static_cast<int64_t>(kBlockThreads) * (dt == STAR_DTYPE_BF16 ? kVecBF16 : kVecF32);
}

// The workspace is sized for the smaller (fp32) tile, i.e. the larger tile
// count, so that its size does not depend on the gradient dtype, plus one tile
// per tensor for leading elements in front of a vector-aligned body.
constexpr int64_t kTileForSizing = static_cast<int64_t>(kBlockThreads) * kVecF32;

size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct WorkspaceLayout {
    size_t tensors_off, grads_off, snaps_off, tiles_off, total;
};

WorkspaceLayout layout_for(int n_tensors, int W, int n_sets, int64_t n_tiles)
{
    const size_t T = static_cast<size_t>(n_tensors);
    WorkspaceLayout l;
    l.tensors_off = 0;
    l.grads_off = round_up(l.tensors_off + sizeof(TensorEntry) * T, kWorkspaceAlign);
    l.snaps_off = round_up(l.grads_off + sizeof(void *) * T * static_cast<size_t>(W), kWorkspaceAlign);
    l.tiles_off = round_up(l.snaps_off + sizeof(void *) * T * static_cast<size_t>(n_sets), kWorkspaceAlign);
    l.total = round_up(l.tiles_off + sizeof(int32_t) * static_cast<size_t>(n_tiles), kWorkspaceAlign);
    if (l.total == 0) l.total = kWorkspaceAlign;
    return l;
}

star_status_t count_tiles(int n_tensors, const int64_t *sizes, int64_t tile, int64_t *n_tiles, int64_t *total)
{
    *n_tiles = 0;
    *total = 0;
    for (int t = 0; t < n_tensors; ++t) {
        if (sizes[t] < 0) return STAR_ERR_INVALID_ARG;
        *n_tiles += (sizes[t] + tile - 1) / tile + (sizes[t] > 0 ? 1 : 0);
        *total += sizes[t];
    }
    return STAR_OK;
}

// No buffer that the round writes (p, v, snapshots) may share memory with any
// other buffer of the list: different blocks update different tensors at the
// same time.  Gradients are only read and may alias one another.
struct Interval {
    uintptr_t begin, end;
    bool written;
};

bool written_buffers_are_disjoint(std::vector<Interval> &iv)
{
    std::sort(iv.begin(), iv.end(), [](const Interval &a, const Interval &b) { return a.begin < b.begin; });
    uintptr_t end_any = 0, end_written = 0;
    for (const Interval &x : iv) {
        if (x.begin < (x.written ? end_any : end_written)) return false;
        end_any = std::max(end_any, x.end);
        if (x.written) end_written = std::max(end_written, x.end);
    }
    return true;
}

// The prepare calls copy from a host buffer that is released on return: inside
// a stream capture that copy would be replayed from freed memory.
star_status_t refuse_capture(cudaStream_t stream)
{
    cudaStreamCaptureStatus status = cudaStreamCaptureStatusNone;
    const cudaError_t e = cudaStreamIsCapturing(stream, &status);
    if (e != cudaSuccess) return cuda_failed(e);
    return status == cudaStreamCaptureStatusNone ? STAR_OK : STAR_ERR_UNSUPPORTED;
}

star_status_t multi_prepare(int n_tensors, float *const *params, float *const *momentum,
                            const void *const *grads, const int64_t *sizes, int W, star_dtype_t grad_dtype,
                            int n_sets, void *const *snapshots, star_dtype_t snapshot_dtype,
                            void *d_workspace, size_t workspace_bytes, void *cuda_stream,
                            star_multi_plan_t *plan_out)
{
    if (!plan_out) return STAR_ERR_NULL_POINTER;
    std::memset(plan_out, 0, sizeof *plan_out);
    if (n_tensors < 0 || W < 0 || n_sets < 0) return STAR_ERR_INVALID_ARG;
    if (grad_dtype != STAR_DTYPE_F32 && grad_dtype != STAR_DTYPE_BF16) return STAR_ERR_INVALID_ARG;
    if (snapshot_dtype != STAR_DTYPE_F32 && snapshot_dtype != STAR_DTYPE_BF16) return STAR_ERR_INVALID_ARG;
    if (W > STAR_MAX_WORKERS || n_sets > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    if (n_tensors > 0 && (!params || !momentum || !grads || !sizes)) return STAR_ERR_NULL_POINTER;
    if (n_tensors > 0 && n_sets > 0 && !snapshots) return STAR_ERR_NULL_POINTER;
    if (!d_workspace) return STAR_ERR_NULL_POINTER;
    if (!aligned(d_workspace, kWorkspaceAlign)) return STAR_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    star_status_t st = refuse_capture(stream);
    if (st != STAR_OK) return st;

    const int64_t tile = tile_elements(grad_dtype);
    const int full_vec = grad_dtype == STAR_DTYPE_BF16 ? kVecBF16 : kVecF32;
    int64_t sizing_tiles = 0, total = 0;
    st = count_tiles(n_tensors, sizes, kTileForSizing, &sizing_tiles, &total);
    if (st != STAR_OK) return st;
    const WorkspaceLayout l = layout_for(n_tensors, W, n_sets, sizing_tiles);
    if (workspace_bytes < l.total) return STAR_ERR_WORKSPACE_TOO_SMALL;

    const unsigned gsize = grad_dtype == STAR_DTYPE_BF16 ? 2 : 4;
    const unsigned snap_elem = snapshot_dtype == STAR_DTYPE_BF16 ? 2 : 4;
    uint64_t complete = W == 64 ? ~uint64_t{0} : ((uint64_t{1} << W) - 1);
    std::vector<unsigned char> host(l.total, 0);
    std::vector<Interval> intervals;
    intervals.reserve(static_cast<size_t>(n_tensors) * static_cast<size_t>(2 + W + n_sets));
    TensorEntry *entries = reinterpret_cast<TensorEntry *>(host.data() + l.tensors_off);
    const void **table = reinterpret_cast<const void **>(host.data() + l.grads_off);
    void **snap_table = reinterpret_cast<void **>(host.data() + l.snaps_off);
    int32_t *tile_tensor = reinterpret_cast<int32_t *>(host.data() + l.tiles_off);
    int64_t next_tile = 0;
    for (int t = 0; t < n_tensors; ++t) {
        const int64_t size = sizes[t];
        TensorEntry &e = entries[t];
        e.params = params[t];
        e.momentum = momentum[t];
        e.size = size;
        e.first_tile = next_tile;
        Buffers buffers;
        auto note = [&](const void *ptr, unsigned elem, bool written) {
            const uintptr_t a = reinterpret_cast<uintptr_t>(ptr);
            intervals.push_back(Interval{a, a + static_cast<uintptr_t>(size) * elem, written});
            buffers.add(ptr, elem);
        };
        if (size > 0) {
            if (!params[t] || !momentum[t]) return STAR_ERR_NULL_POINTER;
            if (!aligned(params[t], 4) || !aligned(momentum[t], 4)) return STAR_ERR_INVALID_ARG;
            note(params[t], 4, true);
            note(momentum[t], 4, true);
        }
        for (int w = 0; w < W; ++w) {
            const void *g = grads[static_cast<size_t>(t) * W + w];
            table[static_cast<size_t>(t) * W + w] = g;
            if (size == 0) continue;
            if (!g) {
                complete &= ~(uint64_t{1} << w);
                continue;
            }
            if (!aligned(g, gsize)) return STAR_ERR_INVALID_ARG;
            note(g, gsize, false);
        }
        for (int set = 0; set < n_sets; ++set) {
            void *snap = snapshots[static_cast<size_t>(t) * n_sets + set];
            snap_table[static_cast<size_t>(t) * n_sets + set] = snap;
            if (size == 0 || !snap) continue;
            if (!aligned(snap, snap_elem)) return STAR_ERR_INVALID_ARG;
            note(snap, snap_elem, true);
        }
        const VectorPlan plan = plan_vector(grad_dtype, buffers, size, false);
        e.vec = plan.vec == full_vec ? full_vec : 1;
        e.head = e.vec == full_vec ? plan.head : 0;
        const int64_t tiles_here = (size - e.head + tile - 1) / tile + (e.head > 0 ? 1 : 0);
        for (int64_t i = 0; i < tiles_here; ++i) tile_tensor[next_tile + i] = t;
        next_tile += tiles_here;
    }
    if (!written_buffers_are_disjoint(intervals)) return STAR_ERR_INVALID_ARG;

    const size_t used = round_up(l.tiles_off + sizeof(int32_t) * static_cast<size_t>(next_tile), kWorkspaceAlign);
    const cudaError_t e = cudaMemcpyAsync(d_workspace, host.data(), std::min(used, l.total), cudaMemcpyHostToDevice,
                                          stream);
    if (e != cudaSuccess) return cuda_failed(e);

    plan_out->magic = kPlanMagic;
    plan_out->d_workspace = d_workspace;
    plan_out->total_elements = total;
    plan_out->n_tiles = next_tile;
    plan_out->complete_workers = complete;
    plan_out->n_tensors = n_tensors;
    plan_out->W = W;
    plan_out->grad_dtype = static_cast<int32_t>(grad_dtype);
    plan_out->tile_elements = static_cast<int32_t>(tile);
    plan_out->n_snapshot_sets = n_sets;
    plan_out->snapshot_dtype = static_cast<int32_t>(snapshot_dtype);
    return STAR_OK;
}

}  // namespace

extern "C" star_status_t star_multi_workspace_bytes_ex(int n_tensors, const int64_t *sizes, int W,
                                                       int n_snapshot_sets, size_t *bytes_out)
{
    if (!bytes_out) return STAR_ERR_NULL_POINTER;
    if (n_tensors < 0 || W < 0 || n_snapshot_sets < 0) return STAR_ERR_INVALID_ARG;
    if (W > STAR_MAX_WORKERS || n_snapshot_sets > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    if (n_tensors > 0 && !sizes) return STAR_ERR_NULL_POINTER;
    int64_t n_tiles = 0, total = 0;
    const star_status_t st = count_tiles(n_tensors, sizes, kTileForSizing, &n_tiles, &total);
    if (st != STAR_OK) return st;
    *bytes_out = layout_for(n_tensors, W, n_snapshot_sets, n_tiles).total;
    return STAR_OK;
}

extern "C" star_status_t star_multi_workspace_bytes(int n_tensors, const int64_t *sizes, int W,
                                                    size_t *bytes_out)
{
    return star_multi_workspace_bytes_ex(n_tensors, sizes, W, 0, bytes_out);
}

extern "C" star_status_t star_multi_prepare(int n_tensors, float *const *params, float *const *momentum,
                                            const void *const *grads, const int64_t *sizes, int W,
                                            star_dtype_t grad_dtype, void *d_workspace,
                                            size_t workspace_bytes, void *cuda_stream,
                                            star_multi_plan_t *plan_out)
{
    return multi_prepare(n_tensors, params, momentum, grads, sizes, W, grad_dtype, 0, nullptr, STAR_DTYPE_F32,
                         d_workspace, workspace_bytes, cuda_stream, plan_out);
}

extern "C" star_status_t star_multi_prepare_ex(int n_tensors, float *const *params, float *const *momentum,
                                               const void *const *grads, const int64_t *sizes, int W,
                                               star_dtype_t grad_dtype, int n_snapshot_sets,
                                               void *const *snapshots, star_dtype_t snapshot_dtype,
                                               void *d_workspace, size_t workspace_bytes, void *cuda_stream,
                                               star_multi_plan_t *plan_out)
{
    return multi_prepare(n_tensors, params, momentum, grads, sizes, W, grad_dtype, n_snapshot_sets, snapshots,
                         snapshot_dtype, d_workspace, workspace_bytes, cuda_stream, plan_out);
}

namespace {

template <typename Kernel, typename Args>
star_status_t launch_tiles(Kernel kernel, Geometry *cache, const Args &args, int64_t n_tiles, cudaStream_t stream)
{
    int blocks = 0;
    cudaError_t e = resident_blocks(kernel, cache, &blocks);
    if (e != cudaSuccess) return cuda_failed(e);
    // The tile-map kernel pays a table lookup per block: measured on B200 the
    // persistent grid is the faster shape for it at every list size tried.
    const int grid = static_cast<int>(n_tiles < blocks ? n_tiles : blocks);
    kernel<<<grid, kBlockThreads, 0, stream>>>(args);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_failed(e);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return STAR_OK;
}

template <typename G, int VEC>
star_status_t launch_multi(const MultiArgs &args, cudaStream_t stream)
{
    static Geometry cache[kMaxDevices];
    return launch_tiles(star_update_multi_kernel<G, VEC, kDepthVector>, cache, args, args.n_tiles, stream);
}

template <typename G, int VEC, int TREE>
star_status_t launch_multi_ex(const MultiExArgs &args, cudaStream_t stream)
{
    static Geometry cache[kMaxDevices];
    return launch_tiles(star_update_multi_ex_kernel<G, VEC, kDepthVector, TREE>, cache, args, args.base.n_tiles,
                        stream);
}

template <typename G, int VEC>
star_status_t dispatch_multi_ex(const MultiExArgs &args, int tree, cudaStream_t stream)
{
    switch (tree) {
    case 4: return launch_multi_ex<G, VEC, 4>(args, stream);
    case 16: return launch_multi_ex<G, VEC, 16>(args, stream);
    case 64: return launch_multi_ex<G, VEC, 64>(args, stream);
    default: return launch_multi_ex<G, VEC, 0>(args, stream);
    }
}

// One round over a prepared list.  snapshot_set_of_group == nullptr and the
// linear order take the plain kernel.
star_status_t update_multi(const star_multi_plan_t *plan, const int32_t *group_offsets,
                           const int32_t *group_members, int n_groups, float lr, const float *lrs, float mu,
                           float wd, const int32_t *snapshot_set_of_group, star_sum_order_t sum_order,
                           void *cuda_stream)
{
    if (!plan) return STAR_ERR_NULL_POINTER;
    if (plan->magic != kPlanMagic || !plan->d_workspace) return STAR_ERR_INVALID_ARG;
    if (sum_order != STAR_SUM_LINEAR && sum_order != STAR_SUM_TREE) return STAR_ERR_INVALID_ARG;
    MultiExArgs ex;
    MultiArgs &args = ex.base;
    const star_status_t st = flatten_schedule(group_offsets, group_members, n_groups, plan->W, lr, &args.sched, lrs);
    if (st != STAR_OK) return st;
    bool any_snapshot = false;
    std::memset(ex.snapshot_set, -1, sizeof ex.snapshot_set);
    for (int k = 0; snapshot_set_of_group && k < n_groups; ++k) {
        const int set = snapshot_set_of_group[k];
        if (set < -1 || set >= plan->n_snapshot_sets) return STAR_ERR_INVALID_ARG;
        if (set < 0) continue;
        ex.snapshot_set[group_offsets[k + 1] - 1] = static_cast<int8_t>(set);
        any_snapshot = true;
    }
    if (plan->n_tiles == 0 || n_groups == 0) return STAR_OK;
    for (int j = 0; j < args.sched.n_slots; ++j)
        if (!(plan->complete_workers >> args.sched.member[j] & 1u)) return STAR_ERR_NULL_POINTER;

    const star_dtype_t dt = static_cast<star_dtype_t>(plan->grad_dtype);
    if (dt != STAR_DTYPE_BF16 && dt != STAR_DTYPE_F32) return STAR_ERR_INVALID_ARG;
    // the offsets of the tables do not depend on the number of tiles
    const WorkspaceLayout l = layout_for(plan->n_tensors, plan->W, plan->n_snapshot_sets, plan->n_tiles);
    const char *base = static_cast<const char *>(plan->d_workspace);
    args.tensors = reinterpret_cast<const TensorEntry *>(base + l.tensors_off);
    args.grads = reinterpret_cast<const void *const *>(base + l.grads_off);
    args.tile_tensor = reinterpret_cast<const int32_t *>(base + l.tiles_off);
    args.n_tiles = plan->n_tiles;
    args.W = plan->W;
    args.hyper = Hyper{mu, wd};
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int tree = tree_span(sum_order, largest_group(group_offsets, n_groups));
    if (tree == 0 && !any_snapshot)
        return dt == STAR_DTYPE_BF16 ? launch_multi<GradBF16, kVecBF16>(args, stream)
                                     : launch_multi<GradF32, kVecF32>(args, stream);
    ex.snapshots = reinterpret_cast<void *const *>(base + l.snaps_off);
    ex.n_sets = plan->n_snapshot_sets;
    ex.snapshot_bf16 = plan->snapshot_dtype == STAR_DTYPE_BF16 ? 1 : 0;
    return dt == STAR_DTYPE_BF16 ? dispatch_multi_ex<GradBF16, kVecBF16>(ex, tree, stream)
                                 : dispatch_multi_ex<GradF32, kVecF32>(ex, tree, stream);
}

}  // namespace

extern "C" star_status_t star_group_update_multi(const star_multi_plan_t *plan,
                                                 const int32_t *group_offsets, const int32_t *group_members,
                                                 int n_groups, float lr, float mu, float wd,
                                                 void *cuda_stream)
{
    return update_multi(plan, group_offsets, group_members, n_groups, lr, nullptr, mu, wd, nullptr, STAR_SUM_LINEAR,
                        cuda_stream);
}

extern "C" star_status_t star_group_update_multi_lrs(const star_multi_plan_t *plan,
                                                     const int32_t *group_offsets,
                                                     const int32_t *group_members, int n_groups,
                                                     const float *lrs, float mu, float wd, void *cuda_stream)
{
    if (n_groups > 0 && !lrs) return STAR_ERR_NULL_POINTER;
    return update_multi(plan, group_offsets, group_members, n_groups, 0.0f, lrs, mu, wd, nullptr, STAR_SUM_LINEAR,
                        cuda_stream);
}

extern "C" star_status_t star_group_update_multi_ex(const star_multi_plan_t *plan,
                                                    const int32_t *group_offsets,
                                                    const int32_t *group_members, int n_groups,
                                                    const float *lrs, float mu, float wd,
                                                    const int32_t *snapshot_set_of_group,
                                                    star_sum_order_t sum_order, void *cuda_stream)
{
    if (n_groups > 0 && !lrs) return STAR_ERR_NULL_POINTER;
    return update_multi(plan, group_offsets, group_members, n_groups, 0.0f, lrs, mu, wd, snapshot_set_of_group,
                        sum_order, cuda_stream);
}

// ---------------------------------------------------------------------------
// Host-resident state and gradients: chunked, double-buffered streaming.
// ---------------------------------------------------------------------------
namespace {

constexpr int64_t kHostChunkQuantum = 2048;

struct HostPipeline {            // per device, created on first use, never destroyed
    cudaStream_t copy_back = nullptr;
    cudaEvent_t kernel_done[2] = {nullptr, nullptr};
    cudaEvent_t copied_back[2] = {nullptr, nullptr};
    bool ready = false;
};

std::mutex g_host_mutex[kMaxDevices];
HostPipeline g_host_pipeline[kMaxDevices];

cudaError_t host_pipeline(int dev, HostPipeline **out)
{
    HostPipeline &hp = g_host_pipeline[dev];
    if (!hp.ready) {
        cudaError_t e = cudaStreamCreateWithFlags(&hp.copy_back, cudaStreamNonBlocking);
        if (e != cudaSuccess) return e;
        for (int i = 0; i < 2; ++i) {
            e = cudaEventCreateWithFlags(&hp.kernel_done[i], cudaEventDisableTiming);
            if (e != cudaSuccess) return e;
            e = cudaEventCreateWithFlags(&hp.copied_back[i], cudaEventDisableTiming);
            if (e != cudaSuccess) return e;
        }
        hp.ready = true;
    }
    *out = &hp;
    return cudaSuccess;
}

// Bytes of one staging set (p, v, `scheduled` gradient chunks and `snapshots`
// snapshot chunks), each sub-buffer rounded up to the workspace alignment.
size_t host_set_bytes(int scheduled, size_t gsize, int snapshots, size_t ssize, int64_t chunk)
{
    const size_t state = round_up(static_cast<size_t>(chunk) * 4, kWorkspaceAlign);
    const size_t grad = round_up(static_cast<size_t>(chunk) * gsize, kWorkspaceAlign);
    const size_t snap = round_up(static_cast<size_t>(chunk) * ssize, kWorkspaceAlign);
    return 2 * state + static_cast<size_t>(scheduled) * grad + static_cast<size_t>(snapshots) * snap;
}

// The host-buffer round: chunked, double-buffered.  lrs == nullptr: one rate lr.
star_status_t host_update(float *h_params, float *h_momentum, const void *const *h_grads, int W,
                          star_dtype_t grad_dtype, int64_t n, const int32_t *group_offsets,
                          const int32_t *group_members, int n_groups, float lr, const float *lrs, float mu, float wd,
                          void *const *h_snapshots, star_dtype_t snapshot_dtype, star_sum_order_t sum_order,
                          void *d_workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (n < 0 || W < 0) return STAR_ERR_INVALID_ARG;
    if (grad_dtype != STAR_DTYPE_F32 && grad_dtype != STAR_DTYPE_BF16) return STAR_ERR_INVALID_ARG;
    if (snapshot_dtype != STAR_DTYPE_F32 && snapshot_dtype != STAR_DTYPE_BF16) return STAR_ERR_INVALID_ARG;
    if (sum_order != STAR_SUM_LINEAR && sum_order != STAR_SUM_TREE) return STAR_ERR_INVALID_ARG;
    if (W > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    SnapshotArgs sargs;
    FlatArgs &args = sargs.flat;
    const star_status_t st = flatten_schedule(group_offsets, group_members, n_groups, W, lr, &args.sched, lrs);
    if (st != STAR_OK) return st;
    if (n == 0 || n_groups == 0) return STAR_OK;
    if (!h_params || !h_momentum || !h_grads || !d_workspace) return STAR_ERR_NULL_POINTER;
    if (!aligned(d_workspace, kWorkspaceAlign)) return STAR_ERR_INVALID_ARG;

    const size_t gsize = grad_dtype == STAR_DTYPE_BF16 ? 2 : 4;
    const size_t ssize = snapshot_dtype == STAR_DTYPE_BF16 ? 2 : 4;
    const int scheduled = args.sched.n_slots;
    const size_t state_bytes = static_cast<size_t>(n) * 4, grad_bytes = static_cast<size_t>(n) * gsize;
    const size_t snap_bytes = static_cast<size_t>(n) * ssize;
    if (!aligned(h_params, 4) || !aligned(h_momentum, 4)) return STAR_ERR_INVALID_ARG;
    if (overlaps(h_params, state_bytes, h_momentum, state_bytes)) return STAR_ERR_INVALID_ARG;
    for (int j = 0; j < scheduled; ++j) {
        const void *g = h_grads[args.sched.member[j]];
        if (!g) return STAR_ERR_NULL_POINTER;
        if (!aligned(g, gsize)) return STAR_ERR_INVALID_ARG;
        if (overlaps(g, grad_bytes, h_params, state_bytes) || overlaps(g, grad_bytes, h_momentum, state_bytes))
            return STAR_ERR_INVALID_ARG;
    }
    // Snapshots: closing slot of the group and host destination, in group order.
    int snap_slot[STAR_MAX_WORKERS];
    void *snap_host[STAR_MAX_WORKERS];
    int n_snap = 0;
    for (int k = 0; h_snapshots && k < n_groups; ++k) {
        void *snap = h_snapshots[k];
        if (!snap) continue;
        if (!aligned(snap, ssize)) return STAR_ERR_INVALID_ARG;
        if (overlaps(snap, snap_bytes, h_params, state_bytes) || overlaps(snap, snap_bytes, h_momentum, state_bytes))
            return STAR_ERR_INVALID_ARG;
        for (int j = 0; j < scheduled; ++j)
            if (overlaps(snap, snap_bytes, h_grads[args.sched.member[j]], grad_bytes)) return STAR_ERR_INVALID_ARG;
        for (int l = 0; l < n_snap; ++l)
            if (overlaps(snap, snap_bytes, snap_host[l], snap_bytes)) return STAR_ERR_INVALID_ARG;
        snap_slot[n_snap] = group_offsets[k + 1] - 1;
        snap_host[n_snap] = snap;
        ++n_snap;
    }
    const int tree = tree_span(sum_order, largest_group(group_offsets, n_groups));
    const bool extended = tree != 0 || n_snap > 0;

    // Largest chunk (multiple of the quantum) whose two staging sets fit.
    const size_t per_element = 8 + static_cast<size_t>(scheduled) * gsize + static_cast<size_t>(n_snap) * ssize;
    int64_t chunk = static_cast<int64_t>(workspace_bytes / (2 * per_element));
    chunk = chunk / kHostChunkQuantum * kHostChunkQuantum;
    while (chunk >= kHostChunkQuantum && 2 * host_set_bytes(scheduled, gsize, n_snap, ssize, chunk) > workspace_bytes)
        chunk -= kHostChunkQuantum;
    if (chunk < kHostChunkQuantum) return STAR_ERR_WORKSPACE_TOO_SMALL;
    const int64_t needed = (n + kHostChunkQuantum - 1) / kHostChunkQuantum * kHostChunkQuantum;
    if (chunk > needed) chunk = needed;

    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_failed(e);
    if (dev < 0 || dev >= kMaxDevices) return cuda_failed(cudaErrorInvalidDevice);
    std::lock_guard<std::mutex> lock(g_host_mutex[dev]);
    HostPipeline *hp = nullptr;
    e = host_pipeline(dev, &hp);
    if (e != cudaSuccess) return cuda_failed(e);

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t set_bytes = host_set_bytes(scheduled, gsize, n_snap, ssize, chunk);
    const size_t state_stride = round_up(static_cast<size_t>(chunk) * 4, kWorkspaceAlign);
    const size_t grad_stride = round_up(static_cast<size_t>(chunk) * gsize, kWorkspaceAlign);
    const size_t snap_stride = round_up(static_cast<size_t>(chunk) * ssize, kWorkspaceAlign);
    char *const base = static_cast<char *>(d_workspace);
    args.hyper = Hyper{mu, wd};
    args.head = 0;
    sargs.snapshot_bf16 = snapshot_dtype == STAR_DTYPE_BF16 ? 1 : 0;
    // staging buffers are aligned: full vector width, no leading elements
    const VectorPlan plan{grad_dtype == STAR_DTYPE_BF16 ? kVecBF16 : kVecF32, 0};

    // The staging sets may still be in use by an earlier call's copy-back
    // (another stream): order this call's first writes after it.
    for (int b = 0; b < 2; ++b) {
        e = cudaStreamWaitEvent(stream, hp->copied_back[b], 0);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    int64_t index = 0;
    for (int64_t first = 0; first < n; first += chunk, ++index) {
        const int b = static_cast<int>(index & 1);
        const int64_t count = n - first < chunk ? n - first : chunk;
        char *set = base + static_cast<size_t>(b) * set_bytes;
        float *d_p = reinterpret_cast<float *>(set);
        float *d_v = reinterpret_cast<float *>(set + state_stride);
        char *d_grads = set + 2 * state_stride;
        char *d_snaps = d_grads + static_cast<size_t>(scheduled) * grad_stride;
        if (index >= 2) {                       // set b was last used by chunk index - 2
            e = cudaStreamWaitEvent(stream, hp->copied_back[b], 0);
            if (e != cudaSuccess) return cuda_failed(e);
        }
        e = cudaMemcpyAsync(d_p, h_params + first, static_cast<size_t>(count) * 4, cudaMemcpyHostToDevice, stream);
        if (e != cudaSuccess) return cuda_failed(e);
        e = cudaMemcpyAsync(d_v, h_momentum + first, static_cast<size_t>(count) * 4, cudaMemcpyHostToDevice, stream);
        if (e != cudaSuccess) return cuda_failed(e);
        std::memset(args.grads, 0, sizeof args.grads);
        for (int j = 0; j < scheduled; ++j) {
            const int w = args.sched.member[j];
            char *d_g = d_grads + static_cast<size_t>(j) * grad_stride;
            const char *h_g = static_cast<const char *>(h_grads[w]) + static_cast<size_t>(first) * gsize;
            e = cudaMemcpyAsync(d_g, h_g, static_cast<size_t>(count) * gsize, cudaMemcpyHostToDevice, stream);
            if (e != cudaSuccess) return cuda_failed(e);
            args.grads[w] = d_g;
        }
        std::memset(sargs.snapshots, 0, sizeof sargs.snapshots);
        for (int l = 0; l < n_snap; ++l) sargs.snapshots[snap_slot[l]] = d_snaps + static_cast<size_t>(l) * snap_stride;
        args.params = d_p;
        args.momentum = d_v;
        args.n = count;
        const star_status_t ls = extended ? dispatch_extended(sargs, grad_dtype, plan, tree, stream)
                                          : dispatch_flat(args, grad_dtype, plan, stream);
        if (ls != STAR_OK) return ls;
        e = cudaEventRecord(hp->kernel_done[b], stream);
        if (e != cudaSuccess) return cuda_failed(e);
        e = cudaStreamWaitEvent(hp->copy_back, hp->kernel_done[b], 0);
        if (e != cudaSuccess) return cuda_failed(e);
        e = cudaMemcpyAsync(h_params + first, d_p, static_cast<size_t>(count) * 4, cudaMemcpyDeviceToHost, hp->copy_back);
        if (e != cudaSuccess) return cuda_failed(e);
        e = cudaMemcpyAsync(h_momentum + first, d_v, static_cast<size_t>(count) * 4, cudaMemcpyDeviceToHost, hp->copy_back);
        if (e != cudaSuccess) return cuda_failed(e);
        for (int l = 0; l < n_snap; ++l) {
            char *h_s = static_cast<char *>(snap_host[l]) + static_cast<size_t>(first) * ssize;
            e = cudaMemcpyAsync(h_s, d_snaps + static_cast<size_t>(l) * snap_stride, static_cast<size_t>(count) * ssize,
                                cudaMemcpyDeviceToHost, hp->copy_back);
            if (e != cudaSuccess) return cuda_failed(e);
        }
        e = cudaEventRecord(hp->copied_back[b], hp->copy_back);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    // Later work on the caller's stream (and its synchronize) sees the results.
    for (int b = 0; b < 2; ++b) {
        e = cudaStreamWaitEvent(stream, hp->copied_back[b], 0);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    return STAR_OK;
}

}  // namespace

extern "C" star_status_t star_host_workspace_bytes_ex(int max_scheduled, star_dtype_t grad_dtype,
                                                      int max_snapshots, star_dtype_t snapshot_dtype,
                                                      int64_t chunk_elements, size_t *bytes_out)
{
    if (!bytes_out) return STAR_ERR_NULL_POINTER;
    if (grad_dtype != STAR_DTYPE_F32 && grad_dtype != STAR_DTYPE_BF16) return STAR_ERR_INVALID_ARG;
    if (snapshot_dtype != STAR_DTYPE_F32 && snapshot_dtype != STAR_DTYPE_BF16) return STAR_ERR_INVALID_ARG;
    if (max_scheduled < 0 || max_snapshots < 0 || chunk_elements < kHostChunkQuantum ||
        chunk_elements % kHostChunkQuantum != 0)
        return STAR_ERR_INVALID_ARG;
    if (max_scheduled > STAR_MAX_WORKERS || max_snapshots > STAR_MAX_WORKERS) return STAR_ERR_UNSUPPORTED;
    *bytes_out = 2 * host_set_bytes(max_scheduled, grad_dtype == STAR_DTYPE_BF16 ? 2 : 4, max_snapshots,
                                    snapshot_dtype == STAR_DTYPE_BF16 ? 2 : 4, chunk_elements);
    return STAR_OK;
}

extern "C" star_status_t star_host_workspace_bytes(int max_scheduled, star_dtype_t grad_dtype,
                                                   int64_t chunk_elements, size_t *bytes_out)
{
    return star_host_workspace_bytes_ex(max_scheduled, grad_dtype, 0, STAR_DTYPE_F32, chunk_elements, bytes_out);
}

extern "C" star_status_t star_group_update_host(float *h_params, float *h_momentum,
                                                const void *const *h_grads, int W,
                                                star_dtype_t grad_dtype, int64_t n,
                                                const int32_t *group_offsets,
                                                const int32_t *group_members, int n_groups, float lr,
                                                float mu, float wd, void *d_workspace,
                                                size_t workspace_bytes, void *cuda_stream)
{
    return host_update(h_params, h_momentum, h_grads, W, grad_dtype, n, group_offsets, group_members, n_groups, lr,
                       nullptr, mu, wd, nullptr, STAR_DTYPE_F32, STAR_SUM_LINEAR, d_workspace, workspace_bytes,
                       cuda_stream);
}

extern "C" star_status_t star_group_update_host_ex(float *h_params, float *h_momentum,
                                                   const void *const *h_grads, int W,
                                                   star_dtype_t grad_dtype, int64_t n,
                                                   const int32_t *group_offsets,
                                                   const int32_t *group_members, int n_groups,
                                                   const float *lrs, float mu, float wd,
                                                   void *const *h_snapshots, star_dtype_t snapshot_dtype,
                                                   star_sum_order_t sum_order, void *d_workspace,
                                                   size_t workspace_bytes, void *cuda_stream)
{
    if (n_groups > 0 && !lrs) return STAR_ERR_NULL_POINTER;
    return host_update(h_params, h_momentum, h_grads, W, grad_dtype, n, group_offsets, group_members, n_groups, 0.0f,
                       lrs, mu, wd, h_snapshots, snapshot_dtype, sum_order, d_workspace, workspace_bytes, cuda_stream);
}

// ---------------------------------------------------------------------------
// Tensor-list round without any allocation: the table lives in a fixed array
// of the library's own device image.
// ---------------------------------------------------------------------------
namespace {

// In host code this name is only a handle for the runtime's symbol lookup, not
// an address a kernel could use; the device address comes from
// cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[STAR_STATIC_SCRATCH_BYTES];

std::atomic<void *> g_static_scratch_address[kMaxDevices];

// Device address of the array on the current device, looked up on first use.
cudaError_t static_scratch_address(void **out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    void *ptr = g_static_scratch_address[dev].load(std::memory_order_acquire);
    if (!ptr) {
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        if (!ptr) return cudaErrorInvalidSymbol;
        g_static_scratch_address[dev].store(ptr, std::memory_order_release);   // same value from any thread
    }
    *out = ptr;
    return cudaSuccess;
}

}  // namespace

extern "C" star_status_t star_group_update_multi_noalloc(
    int n_tensors, float *const *params, float *const *momentum, const void *const *grads,
    const int64_t *sizes, int W, star_dtype_t grad_dtype, const int32_t *group_offsets,
    const int32_t *group_members, int n_groups, float lr, float mu, float wd, void *cuda_stream)
{
    // Inside a stream capture nothing is enqueued (the table copy reads host
    // memory that is gone by the time a graph would replay it).
    star_status_t st = refuse_capture(static_cast<cudaStream_t>(cuda_stream));
    if (st != STAR_OK) return st;
    // Reject a bad schedule before the shared table is touched.
    st = star_schedule_validate(group_offsets, group_members, n_groups, W);
    if (st != STAR_OK) return st;
    size_t need = 0;
    st = star_multi_workspace_bytes(n_tensors, sizes, W, &need);
    if (st != STAR_OK) return st;
    if (need > STAR_STATIC_SCRATCH_BYTES) return STAR_ERR_WORKSPACE_TOO_SMALL;
    void *scratch = nullptr;
    const cudaError_t e = static_scratch_address(&scratch);
    if (e != cudaSuccess) return cuda_failed(e);
    // The copy into the array is ordered on cuda_stream after the previous
    // call's kernel and before this call's kernel.
    star_multi_plan_t plan;
    st = star_multi_prepare(n_tensors, params, momentum, grads, sizes, W, grad_dtype, scratch,
                            STAR_STATIC_SCRATCH_BYTES, cuda_stream, &plan);
    if (st != STAR_OK) return st;
    return star_group_update_multi(&plan, group_offsets, group_members, n_groups, lr, mu, wd, cuda_stream);
}
