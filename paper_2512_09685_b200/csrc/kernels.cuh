// Device code of the fused grouped update (sm_100a).
//
// One thread owns VEC consecutive elements of one tensor.  It loads p and v,
// then walks the flattened schedule (all members of all groups, in order) in
// chunks of DEPTH members: the DEPTH gradient loads of a chunk are issued back
// to back before any of them is consumed, so each thread keeps
// DEPTH * 8..16 bytes in flight on top of p and v.  Every group's update is
// applied in registers; p and v are stored once.
//
// The arithmetic is the pinned binary32 sequence
//     s = g_0 + g_1 + ... ; gbar = s / |G| ; d = fma(wd, p, gbar) ;
//     v = fma(mu, v, d)   ; p = fma(-lr, v, p)
// written with round-to-nearest intrinsics, which the compiler neither
// contracts nor reassociates.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace star {

constexpr int kMaxWorkers = 64;
constexpr int kBlockThreads = 256;
// Resident blocks per SM the vector kernels are compiled for: 4 x 256 threads
// at <= 64 registers.  Measured on B200: 32 resident warps per SM with 4 loads
// in flight per thread reach the HBM copy rate; one block of 145-register
// threads (deeper chunks, wider vectors) reached only 63 % of it.
constexpr int kResidentBlocks = 4;

// The schedule as the kernel sees it: one slot per scheduled worker, in the
// order the gradients are consumed.  A slot that closes a group carries that
// group's size and (negated) learning rate.
struct FlatSchedule {
    int32_t n_slots;
    uint8_t member[kMaxWorkers];       // slot -> worker index
    uint8_t group_size[kMaxWorkers];   // |G_k| on the last slot of group k, else 0
    uint8_t index_in_group[kMaxWorkers];   // position of the slot inside its group (tree order only)
    float neg_lr[kMaxWorkers];         // -lr_k on the last slot of group k
};

struct Hyper {
    float mu;
    float wd;
};

// ---------------------------------------------------------------------------
// Memory operations.  Gradients are read exactly once through the read-only
// (non-coherent) path with the default L1 policy: measured on B200 this is
// 2.5-6 % faster than the same loads with L1::no_allocate, evict-first or
// last-use hints (6445 vs 6280 GB/s on the ResNet-50-sized round, 6890 vs 6500
// on the 32-worker ASGD round).  p and v are read once and written once; their
// cache hints made no measurable difference.
// ---------------------------------------------------------------------------
template <int BYTES> struct Raw;              // BYTES of payload in 32-bit registers
template <> struct Raw<2>  { uint32_t w[1]; };
template <> struct Raw<4>  { uint32_t w[1]; };
template <> struct Raw<8>  { uint32_t w[2]; };
template <> struct Raw<16> { uint32_t w[4]; };

template <int BYTES> __device__ __forceinline__ Raw<BYTES> load_stream(const void *p);

template <> __device__ __forceinline__ Raw<2> load_stream<2>(const void *p)
{
    Raw<2> r;
    unsigned short h;
    asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(h) : "l"(p));
    r.w[0] = h;
    return r;
}
template <> __device__ __forceinline__ Raw<4> load_stream<4>(const void *p)
{
    Raw<4> r;
    asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(r.w[0]) : "l"(p));
    return r;
}
template <> __device__ __forceinline__ Raw<8> load_stream<8>(const void *p)
{
    Raw<8> r;
    asm volatile("ld.global.nc.v2.u32 {%0,%1}, [%2];" : "=r"(r.w[0]), "=r"(r.w[1]) : "l"(p));
    return r;
}
template <> __device__ __forceinline__ Raw<16> load_stream<16>(const void *p)
{
    Raw<16> r;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]) : "l"(p));
    return r;
}
// p / v: VEC floats, through 4-, 16- or 32-byte accesses.
template <int VEC> __device__ __forceinline__ void load_state(const float *src, float (&x)[VEC])
{
    if constexpr (VEC == 1) {
        x[0] = *src;
    } else if constexpr (VEC % 8 == 0) {
#pragma unroll
        for (int q = 0; q < VEC / 8; ++q) {
            uint32_t w[8];
            asm volatile("ld.global.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]),
                           "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]) : "l"(src + 8 * q));
#pragma unroll
            for (int e = 0; e < 8; ++e) x[8 * q + e] = __uint_as_float(w[e]);
        }
    } else {
#pragma unroll
        for (int q = 0; q < VEC / 4; ++q) {
            float4 t;
            asm volatile("ld.global.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                         : "=f"(t.x), "=f"(t.y), "=f"(t.z), "=f"(t.w) : "l"(src + 4 * q));
            x[4 * q + 0] = t.x; x[4 * q + 1] = t.y; x[4 * q + 2] = t.z; x[4 * q + 3] = t.w;
        }
    }
}

template <int VEC> __device__ __forceinline__ void store_state(float *dst, const float (&x)[VEC])
{
    if constexpr (VEC == 1) {
        *dst = x[0];
    } else if constexpr (VEC % 8 == 0) {
#pragma unroll
        for (int q = 0; q < VEC / 8; ++q) {
            asm volatile("st.global.L1::no_allocate.v8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"
                         :: "r"(__float_as_uint(x[8 * q + 0])), "r"(__float_as_uint(x[8 * q + 1])),
                            "r"(__float_as_uint(x[8 * q + 2])), "r"(__float_as_uint(x[8 * q + 3])),
                            "r"(__float_as_uint(x[8 * q + 4])), "r"(__float_as_uint(x[8 * q + 5])),
                            "r"(__float_as_uint(x[8 * q + 6])), "r"(__float_as_uint(x[8 * q + 7])),
                            "l"(dst + 8 * q) : "memory");
        }
    } else {
#pragma unroll
        for (int q = 0; q < VEC / 4; ++q) {
            asm volatile("st.global.L1::no_allocate.v4.f32 [%4], {%0,%1,%2,%3};"
                         :: "f"(x[4 * q + 0]), "f"(x[4 * q + 1]), "f"(x[4 * q + 2]),
                            "f"(x[4 * q + 3]), "l"(dst + 4 * q) : "memory");
        }
    }
}

// ---------------------------------------------------------------------------
// Gradient element types.
// ---------------------------------------------------------------------------
struct GradF32 {
    static constexpr int kBytes = 4;
    template <int VEC> static __device__ __forceinline__ void widen(const Raw<VEC * 4> &r, float (&f)[VEC])
    {
#pragma unroll
        for (int e = 0; e < VEC; ++e) f[e] = __uint_as_float(r.w[e]);
    }
};

struct GradBF16 {
    static constexpr int kBytes = 2;
    // bf16 is the upper half of a binary32: widening is a shift / a mask.
    template <int VEC> static __device__ __forceinline__ void widen(const Raw<VEC * 2> &r, float (&f)[VEC])
    {
        if constexpr (VEC == 1) {
            f[0] = __uint_as_float(r.w[0] << 16);
        } else {
#pragma unroll
            for (int e = 0; e < VEC / 2; ++e) {
                f[2 * e + 0] = __uint_as_float(r.w[e] << 16);
                f[2 * e + 1] = __uint_as_float(r.w[e] & 0xffff0000u);
            }
        }
    }
};

// s / count, correctly rounded (IEEE division).  A zero numerator (common:
// gradients of unused embedding rows, dead units, padding) would send the whole
// warp through the division's slow path -- measured 4.2 instead of 6.5 TB/s on
// all-zero gradients -- so zeros are answered directly (+-0 / count = +-0) and
// the division sees a harmless numerator in those lanes.
__device__ __forceinline__ float exact_mean(float s, float count)
{
    const bool zero = s == 0.0f;
    const float q = __fdiv_rn(zero ? 1.0f : s, count);
    return zero ? s : q;
}

// One group update on VEC elements.
template <int VEC>
__device__ __forceinline__ void apply_update(float (&p)[VEC], float (&v)[VEC], const float (&gbar)[VEC],
                                             float neg_lr, const Hyper &h)
{
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
        const float d = __fmaf_rn(h.wd, p[e], gbar[e]);
        v[e] = __fmaf_rn(h.mu, v[e], d);
        p[e] = __fmaf_rn(neg_lr, v[e], p[e]);
    }
}

// All groups of the round on the VEC elements starting at element `first` of
// one tensor.  grad_ptr(slot) returns the base pointer of the slot's worker;
// state_ptr(0) / state_ptr(1) return the tensor's params / momentum base and are
// asked again at store time, so that a caller whose bases live in memory need
// not hold them in registers across the update.
//
// after_group(slot, p) is called right after the update of the group that
// closes on `slot`, with the parameters as they stand then.
struct NoSnapshot {
    template <int VEC> __device__ __forceinline__ void operator()(int, int64_t, const float (&)[VEC]) const {}
};

//
// TREE selects the in-group summation order.  false: left to right.  true:
// pairwise, as along a binary aggregation tree (Section IV-D2b): the partial
// sums pending after i leaves are the set bits of i (level l spans 2^l
// leaves); a new leaf merges with the pending levels below its first clear
// bit, the group's last leaf with every pending level in ascending order.
// That is tree(first h) + tree(rest) with h the largest power of two below the
// group size.  A group of c members needs ceil(log2(c)) pending levels of VEC
// registers each, so the tree kernels are instantiated for 2, 4 and 6 levels
// (groups of up to 4, 16 and 64 members) and compiled for 3, 3 and 2 resident
// blocks; TREE is the number of levels, 0 = linear order.

// Merge a new leaf with the pending partial sums of levels 0..LEVEL-1 and park
// the result on LEVEL.
template <int LEVEL, int VEC, int ROWS>
__device__ __forceinline__ void tree_merge(float (&pending)[ROWS][VEC], float (&f)[VEC])
{
    if constexpr (LEVEL < ROWS) {
#pragma unroll
        for (int l = 0; l < LEVEL; ++l) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) f[e] = __fadd_rn(pending[l][e], f[e]);
        }
#pragma unroll
        for (int e = 0; e < VEC; ++e) pending[LEVEL][e] = f[e];
    }
}

template <typename G, int VEC, int DEPTH, int TREE = 0, typename StatePtr, typename GradPtr,
          typename AfterGroup = NoSnapshot>
__device__ __forceinline__ void update_vector(StatePtr state_ptr, int64_t first, const FlatSchedule &s,
                                              const Hyper &h, GradPtr grad_ptr,
                                              AfterGroup after_group = AfterGroup())
{
    constexpr int GB = VEC * G::kBytes;
    float p[VEC], v[VEC], sum[VEC];
    constexpr int kTreeLevels = TREE;
    [[maybe_unused]] float pending[TREE > 0 ? TREE : 1][VEC];
    load_state<VEC>(state_ptr(0) + first, p);
    load_state<VEC>(state_ptr(1) + first, v);
    // -0.0f is the additive identity of IEEE addition (x + -0 == x for every x,
    // including x == -0), so a running sum started there equals the plain
    // left-to-right sum that starts at the first member.
#pragma unroll
    for (int e = 0; e < VEC; ++e) sum[e] = -0.0f;

    const int n_slots = s.n_slots;
    for (int base = 0; base < n_slots; base += DEPTH) {
        Raw<GB> raw[DEPTH];
#pragma unroll
        for (int j = 0; j < DEPTH; ++j) {
            if (base + j < n_slots) {
                const char *g = static_cast<const char *>(grad_ptr(base + j));
                raw[j] = load_stream<GB>(g + first * G::kBytes);
            }
        }
#pragma unroll
        for (int j = 0; j < DEPTH; ++j) {
            if (base + j < n_slots) {
                float f[VEC];
                G::template widen<VEC>(raw[j], f);
                const int gs = s.group_size[base + j];
                if (gs == 1) {                       // singleton group: the mean is the gradient
                    apply_update<VEC>(p, v, f, s.neg_lr[base + j], h);
                    after_group.template operator()<VEC>(base + j, first, p);
                } else if constexpr (TREE > 0) {
                    const int leaves_before = s.index_in_group[base + j];
                    if (gs == 0) {                   // not the last leaf: merge up to the first clear bit
                        // A real (warp-uniform) branch per level, most frequent level
                        // first: predicating all levels on every leaf made this path
                        // issue-bound, and a jump table was slower than this chain.
                        const int level = __ffs(~leaves_before) - 1;      // number of trailing set bits
                        if (level == 0) {
                            tree_merge<0, VEC>(pending, f);
                        } else if (level == 1) {
                            tree_merge<1, VEC>(pending, f);
                        } else if constexpr (TREE > 2) {
                            if (level == 2) {
                                tree_merge<2, VEC>(pending, f);
                            } else if (level == 3) {
                                tree_merge<3, VEC>(pending, f);
                            } else if constexpr (TREE > 4) {
                                if (level == 4) tree_merge<4, VEC>(pending, f);
                                else tree_merge<5, VEC>(pending, f);
                            }
                        }
                    } else {                         // last leaf: fold every pending level
#pragma unroll
                        for (int l = 0; l < kTreeLevels; ++l) {
                            if (leaves_before >> l & 1) {
#pragma unroll
                                for (int e = 0; e < VEC; ++e) f[e] = __fadd_rn(pending[l][e], f[e]);
                            }
                        }
                        const float count = static_cast<float>(gs);
#pragma unroll
                        for (int e = 0; e < VEC; ++e) f[e] = exact_mean(f[e], count);
                        apply_update<VEC>(p, v, f, s.neg_lr[base + j], h);
                        after_group.template operator()<VEC>(base + j, first, p);
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) sum[e] = __fadd_rn(sum[e], f[e]);
                    if (gs != 0) {
                        const float count = static_cast<float>(gs);
#pragma unroll
                        for (int e = 0; e < VEC; ++e) sum[e] = exact_mean(sum[e], count);
                        apply_update<VEC>(p, v, sum, s.neg_lr[base + j], h);
                        after_group.template operator()<VEC>(base + j, first, p);
#pragma unroll
                        for (int e = 0; e < VEC; ++e) sum[e] = -0.0f;
                    }
                }
            }
        }
    }
    store_state<VEC>(state_ptr(0) + first, p);
    store_state<VEC>(state_ptr(1) + first, v);
}

// ---------------------------------------------------------------------------
// Single flat tensor.
// ---------------------------------------------------------------------------
struct FlatArgs {
    float *params;
    float *momentum;
    const void *grads[kMaxWorkers];
    int64_t n;
    FlatSchedule sched;
    Hyper hyper;
};

// Vector kernel: requires 32-byte aligned bases (p and v move in 32-byte accesses when VEC = 8).
// Grid-stride over vectors; the last < VEC elements are done one by one by the
// first threads of block 0.
template <typename G, int VEC, int DEPTH>
__global__ void __launch_bounds__(kBlockThreads, kResidentBlocks)
star_update_flat_kernel(const __grid_constant__ FlatArgs a)
{
    const int64_t n_vec = a.n / VEC;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kBlockThreads;
    auto grad_ptr = [&](int slot) -> const void * { return a.grads[a.sched.member[slot]]; };
    auto state_ptr = [&](int which) -> float * { return which == 0 ? a.params : a.momentum; };
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kBlockThreads + threadIdx.x; i < n_vec; i += stride)
        update_vector<G, VEC, DEPTH>(state_ptr, i * VEC, a.sched, a.hyper, grad_ptr);
    if constexpr (VEC > 1) {
        const int64_t tail = n_vec * VEC + threadIdx.x;
        if (blockIdx.x == 0 && threadIdx.x < VEC && tail < a.n)
            update_vector<G, 1, DEPTH>(state_ptr, tail, a.sched, a.hyper, grad_ptr);
    }
}

// Flat tensor with the extended options: parameter snapshots (after the update
// of the group that closes on slot j the parameters are also written to
// snapshots[j] if not null -- the copy the server sends back to that group's
// workers) and the tree summation order.
struct SnapshotArgs {
    FlatArgs flat;
    void *snapshots[kMaxWorkers];      // indexed by closing slot; fp32 or bf16 buffers
    int32_t snapshot_bf16;             // 0: snapshots are fp32, 1: rounded to bf16
};

// binary32 -> bf16 bit pattern: round to nearest, ties to even; NaN stays a
// (quiet) NaN.
__device__ __forceinline__ uint32_t narrow_bf16(float f)
{
    uint32_t u = __float_as_uint(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (u >> 16) | 0x0040u;
    u += 0x7fffu + ((u >> 16) & 1u);
    return u >> 16;
}

// VEC parameters as bf16: one 2-, 8- or 16-byte store.
template <int VEC> __device__ __forceinline__ void store_bf16(uint16_t *dst, const float (&x)[VEC])
{
    if constexpr (VEC == 1) {
        *dst = static_cast<uint16_t>(narrow_bf16(x[0]));
    } else {
        uint32_t w[VEC / 2];
#pragma unroll
        for (int e = 0; e < VEC / 2; ++e) w[e] = narrow_bf16(x[2 * e]) | (narrow_bf16(x[2 * e + 1]) << 16);
        if constexpr (VEC == 8) {
            asm volatile("st.global.L1::no_allocate.v4.u32 [%4], {%0,%1,%2,%3};"
                         :: "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "l"(dst) : "memory");
        } else {
            static_assert(VEC == 4, "bf16 snapshot stores exist for 1, 4 and 8 elements");
            asm volatile("st.global.L1::no_allocate.v2.u32 [%2], {%0,%1};" :: "r"(w[0]), "r"(w[1]), "l"(dst) : "memory");
        }
    }
}

struct StoreSnapshot {
    const SnapshotArgs *a;
    template <int VEC> __device__ __forceinline__ void operator()(int slot, int64_t first, const float (&p)[VEC]) const
    {
        void *dst = a->snapshots[slot];
        if (dst == nullptr) return;
        if (a->snapshot_bf16) store_bf16<VEC>(static_cast<uint16_t *>(dst) + first, p);
        else store_state<VEC>(static_cast<float *>(dst) + first, p);
    }
};

constexpr int tree_resident_blocks(int levels)
{
    return levels == 0 ? kResidentBlocks : levels <= 4 ? 3 : 2;
}

template <typename G, int VEC, int DEPTH, int TREE>
__global__ void __launch_bounds__(kBlockThreads, tree_resident_blocks(TREE))
star_update_flat_snapshot_kernel(const __grid_constant__ SnapshotArgs a)
{
    const FlatArgs &f = a.flat;
    const int64_t n_vec = f.n / VEC;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kBlockThreads;
    auto grad_ptr = [&](int slot) -> const void * { return f.grads[f.sched.member[slot]]; };
    auto state_ptr = [&](int which) -> float * { return which == 0 ? f.params : f.momentum; };
    const StoreSnapshot snap{&a};
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kBlockThreads + threadIdx.x; i < n_vec; i += stride)
        update_vector<G, VEC, DEPTH, TREE>(state_ptr, i * VEC, f.sched, f.hyper, grad_ptr, snap);
    if constexpr (VEC > 1) {
        const int64_t tail = n_vec * VEC + threadIdx.x;
        if (blockIdx.x == 0 && threadIdx.x < VEC && tail < f.n)
            update_vector<G, 1, DEPTH, TREE>(state_ptr, tail, f.sched, f.hyper, grad_ptr, snap);
    }
}

// ---------------------------------------------------------------------------
// Tensor list.  The device workspace holds, in this order (each array 256-byte
// aligned): per-tensor TensorEntry records, the gradient pointer table
// [n_tensors * W], and tile_tensor[n_tiles] (tile -> tensor index).  Tiles of a
// tensor are consecutive; TensorEntry::first_tile is the tensor's first tile.
// ---------------------------------------------------------------------------
struct TensorEntry {
    float *params;
    float *momentum;
    int64_t size;          // elements
    int64_t first_tile;
    int32_t vec;           // elements per thread the tensor's buffer alignment allows (full width or less)
    int32_t pad;
};

struct MultiArgs {
    const TensorEntry *tensors;
    const void *const *grads;       // [n_tensors * W]
    const int32_t *tile_tensor;     // [n_tiles]
    int64_t n_tiles;
    int32_t W;
    FlatSchedule sched;
    Hyper hyper;
};

// Element-by-element path for the ragged end of a tensor and for tensors whose
// buffers are not aligned for the full vector width.  Kept out of line: it is
// cold, and inlining it next to the vector path costs registers there.
// Handles elements first, first + step, ... below end.
template <typename G, int DEPTH>
__device__ __noinline__ void update_elements(const TensorEntry &te, const unsigned long long *row,
                                             int64_t first, int64_t end, int64_t step,
                                             const FlatSchedule &s, const Hyper &h)
{
    auto grad_ptr = [&](int slot) -> const void * {
        return reinterpret_cast<const void *>(__ldg(row + s.member[slot]));
    };
    auto state_ptr = [&](int which) -> float * { return which == 0 ? te.params : te.momentum; };
    for (int64_t i = first; i < end; i += step)
        update_vector<G, 1, DEPTH>(state_ptr, i, s, h, grad_ptr);
}

// One block per tile of kBlockThreads * VEC elements (grid-stride over tiles);
// a thread owns one vector of its tile.
template <typename G, int VEC, int DEPTH>
__global__ void __launch_bounds__(kBlockThreads, kResidentBlocks)
star_update_multi_kernel(const __grid_constant__ MultiArgs a)
{
    constexpr int64_t kTile = static_cast<int64_t>(kBlockThreads) * VEC;
    for (int64_t tile = blockIdx.x; tile < a.n_tiles; tile += gridDim.x) {
        const int32_t t = __ldg(a.tile_tensor + tile);
        const TensorEntry &te = a.tensors[t];
        const unsigned long long *row =
            reinterpret_cast<const unsigned long long *>(a.grads) + static_cast<int64_t>(t) * a.W;
        const int64_t begin = (tile - te.first_tile) * kTile;
        const int64_t size = te.size;
        if (te.vec == VEC) {
            const int64_t i = begin + static_cast<int64_t>(threadIdx.x) * VEC;
            if (i + VEC <= size) {
                auto grad_ptr = [&](int slot) -> const void * {
                    return reinterpret_cast<const void *>(__ldg(row + a.sched.member[slot]));
                };
                // Re-read the bases from the (L1-resident) entry instead of
                // keeping four registers live across the update.
                auto state_ptr = [&](int which) -> float * {
                    unsigned long long base;
                    asm volatile("ld.global.nc.u64 %0, [%1];" : "=l"(base)
                                 : "l"(which == 0 ? &te.params : &te.momentum));
                    return reinterpret_cast<float *>(base);
                };
                update_vector<G, VEC, DEPTH>(state_ptr, i, a.sched, a.hyper, grad_ptr);
            } else if (i < size) {                   // the tensor's last, partial vector
                update_elements<G, DEPTH>(te, row, i, size, 1, a.sched, a.hyper);
            }
        } else {
            // Not aligned for the full vector width: element by element.  (A
            // narrower vector path here was measured to cost the aligned path
            // a third of its bandwidth through register spills.)
            const int64_t end = min(size, begin + kTile);
            update_elements<G, DEPTH>(te, row, begin + threadIdx.x, end, kBlockThreads, a.sched, a.hyper);
        }
    }
}

}  // namespace star
