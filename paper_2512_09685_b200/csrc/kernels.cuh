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
// order the gradients are consumed.  A slot that closes a group carries the
// divisor of that group's mean (the group's size; for an update from partial
// sums, the number of gradient reports behind them) and its (negated)
// learning rate; the slot that opens a group carries the group's size for the
// kernels that walk the schedule group by group (tree order).
struct FlatSchedule {
    int32_t n_slots;
    uint8_t member[kMaxWorkers];       // slot -> worker index
    uint8_t group_size[kMaxWorkers];   // divisor of the mean on the last slot of group k, else 0
    uint8_t size_at_start[kMaxWorkers];    // |G_k| on the first slot of group k, else 0
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

// The mean of a group on VEC elements: sum / count, correctly rounded.  For a
// power-of-two count the quotient is the product with the exact reciprocal
// 2^-k -- the same correctly rounded value of the same real number, subnormal
// results, zeros, infinities and NaN included -- which costs one multiply in
// place of the division's ten-odd instructions (groups of 2, 4, 8, 16 are the
// common sizes).  count >= 2.
template <int VEC> __device__ __forceinline__ void mean_rows(float (&sum)[VEC], int count)
{
    if ((count & (count - 1)) == 0) {
        const float inv = __int_as_float((127 - (31 - __clz(count))) << 23);
#pragma unroll
        for (int e = 0; e < VEC; ++e) sum[e] = __fmul_rn(sum[e], inv);
    } else {
        const float c = static_cast<float>(count);
#pragma unroll
        for (int e = 0; e < VEC; ++e) sum[e] = exact_mean(sum[e], c);
    }
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

// after_group(slot, first, p) is called right after the update of the group that
// closes on `slot`, with the parameters as they stand then.
struct NoSnapshot {
    template <int VEC> __device__ __forceinline__ void operator()(int, int64_t, const float (&)[VEC]) const {}
};

template <int VEC> __device__ __forceinline__ void add_rows(float (&a)[VEC], const float (&b)[VEC])
{
#pragma unroll
    for (int e = 0; e < VEC; ++e) a[e] = __fadd_rn(a[e], b[e]);
}

// ---------------------------------------------------------------------------
// Pairwise (tree) summation order, as gradients are combined along a binary
// aggregation tree (Section IV-D2b): tree(m_0..m_{c-1}) is the member itself
// for c = 1, else tree(first h) + tree(remaining c - h) with h the largest
// power of two below c.  Over an aligned span of N = 2^k slots of which the
// first `count` are used that is
//     count <= N/2 : the tree over the first half
//     else         : (full tree over the first half) + (tree over the count - N/2
//                    used slots of the second half)
// so a group is summed by halving with no per-leaf bookkeeping.  Spans of up to
// BLOCK slots are a leaf block: its gradient loads are issued back to back and
// added straight from their registers; each level above a block keeps one
// partial sum (a row of VEC registers).
// ---------------------------------------------------------------------------

// Leaves LO .. LO + N - 1 of a loaded block, of which the first r (1..N) are used.
template <typename G, int VEC, int LO, int N, int BLOCK>
__device__ __forceinline__ void leaf_tree(const Raw<VEC * G::kBytes> (&raw)[BLOCK], int r, float (&out)[VEC])
{
    if constexpr (N == 1) {
        G::template widen<VEC>(raw[LO], out);
    } else {
        constexpr int H = N / 2;
        leaf_tree<G, VEC, LO, H, BLOCK>(raw, min(r, H), out);
        if (r > H) {
            float t[VEC];
            leaf_tree<G, VEC, LO + H, H, BLOCK>(raw, r - H, t);
            add_rows<VEC>(out, t);
        }
    }
}

// Tree-order sum of slots base .. base + count - 1, 1 <= count <= N.
template <typename G, int VEC, int N, int BLOCK, typename GradPtr>
__device__ __forceinline__ void tree_sum(GradPtr grad_ptr, int64_t first, int base, int count, float (&out)[VEC])
{
    if constexpr (N <= BLOCK) {
        constexpr int GB = VEC * G::kBytes;
        Raw<GB> raw[N];
#pragma unroll
        for (int j = 0; j < N; ++j) {
            if (j < count) {
                const char *g = static_cast<const char *>(grad_ptr(base + j));
                raw[j] = load_stream<GB>(g + first * G::kBytes);
            }
        }
        leaf_tree<G, VEC, 0, N, N>(raw, count, out);
    } else {
        constexpr int H = N / 2;
        tree_sum<G, VEC, H, BLOCK>(grad_ptr, first, base, min(count, H), out);
        if (count > H) {
            float t[VEC];
            tree_sum<G, VEC, H, BLOCK>(grad_ptr, first, base + H, count - H, t);
            add_rows<VEC>(out, t);
        }
    }
}

// Leaf block of the tree kernels: the kernel for groups of up to 4 members
// loads a whole group at once and runs at the occupancy of the linear kernels;
// the kernels for larger groups load 8 gradients at a time and run two blocks
// per SM (the rows of partial sums cost registers; the deeper loads keep as
// many bytes in flight per SM).
__host__ __device__ constexpr int tree_block(int tree) { return tree <= 4 ? 4 : 8; }

// Tree-order sum of one group of c <= TREE members whose first slot is `start`.
// Up to two leaf blocks the halving is written out; beyond (groups of up to 64
// members: up to 8 blocks of 8) the blocks are walked by a loop that keeps the
// partial sums of the levels above a block as a binary counter -- after b
// blocks the set bits of b are the pending levels; a new block merges with the
// pending levels below its first clear bit, the last block with every pending
// level in ascending order -- which is the same tree.  (Writing all eight
// blocks out made the compiler hold every gradient pointer in registers.)
template <typename G, int VEC, int TREE, typename GradPtr>
__device__ __forceinline__ void group_tree_sum(GradPtr grad_ptr, int64_t first, int start, int c, float (&out)[VEC])
{
    constexpr int BLOCK = tree_block(TREE);
    if constexpr (TREE <= 2 * BLOCK) {
        tree_sum<G, VEC, TREE, BLOCK>(grad_ptr, first, start, c, out);
    } else {
        static_assert(TREE == 8 * BLOCK, "the block loop keeps three pending levels");
        float pend0[VEC], pend1[VEC], pend2[VEC];
#pragma unroll 1
        for (int b = 0; b * BLOCK < c; ++b) {
            const int left = c - b * BLOCK;
            tree_sum<G, VEC, BLOCK, BLOCK>(grad_ptr, first, start + b * BLOCK, min(left, BLOCK), out);
            if (left > BLOCK) {                      // not the last block: b <= 6
                if ((b & 1) == 0) {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) pend0[e] = out[e];
                } else if ((b & 2) == 0) {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) pend1[e] = __fadd_rn(pend0[e], out[e]);
                } else {                             // b == 3: levels 0 and 1 are pending
#pragma unroll
                    for (int e = 0; e < VEC; ++e) pend2[e] = __fadd_rn(pend1[e], __fadd_rn(pend0[e], out[e]));
                }
            } else {
                if (b & 1) add_rows<VEC>(out, pend0);
                if (b & 2) add_rows<VEC>(out, pend1);
                if (b & 4) add_rows<VEC>(out, pend2);
            }
        }
    }
}

// All groups of the round on the VEC elements starting at element `first` of
// one tensor.  grad_ptr(slot) returns the base pointer of the slot's worker;
// state_ptr(0) / state_ptr(1) return the tensor's params / momentum base and are
// asked again at store time, so that a caller whose bases live in memory need
// not hold them in registers across the update.
//
// TREE = 0: in-group sums run left to right; the flattened schedule is walked
// in chunks of DEPTH slots whatever group they belong to.  TREE = 4, 16 or 64:
// tree order for groups of up to TREE members, walked group by group.
template <typename G, int VEC, int DEPTH, int TREE = 0, typename StatePtr, typename GradPtr,
          typename AfterGroup = NoSnapshot>
__device__ __forceinline__ void update_vector(StatePtr state_ptr, int64_t first, const FlatSchedule &s,
                                              const Hyper &h, GradPtr grad_ptr,
                                              AfterGroup after_group = AfterGroup())
{
    constexpr int GB = VEC * G::kBytes;
    float p[VEC], v[VEC];
    load_state<VEC>(state_ptr(0) + first, p);
    load_state<VEC>(state_ptr(1) + first, v);
    const int n_slots = s.n_slots;

    if constexpr (TREE > 0) {
        for (int start = 0; start < n_slots;) {
            const int c = max(static_cast<int>(s.size_at_start[start]), 1);
            const int closing = start + c - 1;
            float sum[VEC];
            group_tree_sum<G, VEC, TREE>(grad_ptr, first, start, c, sum);
            if (c > 1) mean_rows<VEC>(sum, s.group_size[closing]);
            apply_update<VEC>(p, v, sum, s.neg_lr[closing], h);
            after_group.template operator()<VEC>(closing, first, p);
            start += c;
        }
    } else {
        // -0.0f is the additive identity of IEEE addition (x + -0 == x for every x,
        // including x == -0), so a running sum started there equals the plain
        // left-to-right sum that starts at the first member.
        float sum[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) sum[e] = -0.0f;
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
                    } else {
                        add_rows<VEC>(sum, f);
                        if (gs != 0) {
                            mean_rows<VEC>(sum, gs);
                            apply_update<VEC>(p, v, sum, s.neg_lr[base + j], h);
                            after_group.template operator()<VEC>(base + j, first, p);
#pragma unroll
                            for (int e = 0; e < VEC; ++e) sum[e] = -0.0f;
                        }
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
    int32_t head;          // leading elements (< VEC) done one by one; the vector body starts there
    FlatSchedule sched;
    Hyper hyper;
};

// The elements of a flat tensor that the vector body [head, head + n_vec * VEC)
// leaves over -- up to VEC - 1 in front of it (buffers that are views at an odd
// element offset into aligned storage reach vector alignment only there) and
// up to VEC - 1 behind it -- are done one by one by the first 2 * VEC threads
// of block 0.  Returns the element this thread owns, or -1.
template <int VEC>
__device__ __forceinline__ int64_t edge_element(int64_t n, int head, int64_t n_vec)
{
    if (blockIdx.x != 0 || threadIdx.x >= 2 * VEC) return -1;
    const int t = threadIdx.x;
    if (t < VEC) return t < head ? t : -1;
    const int64_t e = head + n_vec * VEC + (t - VEC);
    return e < n ? e : -1;
}

// Vector kernel: requires bases that are vector-aligned at element `head`
// (32 bytes for p and v when VEC = 8).  Grid-stride over vectors.
template <typename G, int VEC, int DEPTH>
__global__ void __launch_bounds__(kBlockThreads, kResidentBlocks)
star_update_flat_kernel(const __grid_constant__ FlatArgs a)
{
    const int64_t n_vec = (a.n - a.head) / VEC;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kBlockThreads;
    auto grad_ptr = [&](int slot) -> const void * { return a.grads[a.sched.member[slot]]; };
    auto state_ptr = [&](int which) -> float * { return which == 0 ? a.params : a.momentum; };
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kBlockThreads + threadIdx.x; i < n_vec; i += stride)
        update_vector<G, VEC, DEPTH>(state_ptr, a.head + i * VEC, a.sched, a.hyper, grad_ptr);
    if constexpr (VEC > 1) {
        const int64_t e = edge_element<VEC>(a.n, a.head, n_vec);
        if (e >= 0) update_vector<G, 1, DEPTH>(state_ptr, e, a.sched, a.hyper, grad_ptr);
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

// Resident blocks the extended kernels are compiled for: the tree order keeps
// one more row of partial sums per level of four.
constexpr int tree_resident_blocks(int tree)
{
    return tree <= 4 ? kResidentBlocks : 2;
}

template <typename G, int VEC, int DEPTH, int TREE>
__global__ void __launch_bounds__(kBlockThreads, tree_resident_blocks(TREE))
star_update_flat_snapshot_kernel(const __grid_constant__ SnapshotArgs a)
{
    const FlatArgs &f = a.flat;
    const int64_t n_vec = (f.n - f.head) / VEC;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kBlockThreads;
    auto grad_ptr = [&](int slot) -> const void * { return f.grads[f.sched.member[slot]]; };
    auto state_ptr = [&](int which) -> float * { return which == 0 ? f.params : f.momentum; };
    const StoreSnapshot snap{&a};
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kBlockThreads + threadIdx.x; i < n_vec; i += stride)
        update_vector<G, VEC, DEPTH, TREE>(state_ptr, f.head + i * VEC, f.sched, f.hyper, grad_ptr, snap);
    if constexpr (VEC > 1) {
        const int64_t e = edge_element<VEC>(f.n, f.head, n_vec);
        if (e >= 0) update_vector<G, 1, DEPTH, TREE>(state_ptr, e, f.sched, f.hyper, grad_ptr, snap);
    }
}

// ---------------------------------------------------------------------------
// Sum of a list of gradient buffers (all-reduce architecture, Section IV-B: a
// parent adds its children's gradients to its own before the ring): out[i] =
// src[0][i] + src[1][i] + ... in binary32, left to right (TREE = 0) or in tree
// order, stored as binary32 or rounded to bf16.  Every source element is read
// once, every output element written once.
// ---------------------------------------------------------------------------
struct ReduceArgs {
    void *out;
    const void *src[kMaxWorkers];      // in summation order
    int64_t n;
    int32_t count;
    int32_t head;
    int32_t out_bf16;
};

template <typename G, int VEC, int DEPTH, int TREE>
__device__ __forceinline__ void reduce_vector(const ReduceArgs &a, int64_t first)
{
    constexpr int GB = VEC * G::kBytes;
    float sum[VEC];
    auto grad_ptr = [&](int slot) -> const void * { return a.src[slot]; };
    if constexpr (TREE > 0) {
        group_tree_sum<G, VEC, TREE>(grad_ptr, first, 0, a.count, sum);
    } else {
#pragma unroll
        for (int e = 0; e < VEC; ++e) sum[e] = -0.0f;
        for (int base = 0; base < a.count; base += DEPTH) {
            Raw<GB> raw[DEPTH];
#pragma unroll
            for (int j = 0; j < DEPTH; ++j)
                if (base + j < a.count)
                    raw[j] = load_stream<GB>(static_cast<const char *>(a.src[base + j]) + first * G::kBytes);
#pragma unroll
            for (int j = 0; j < DEPTH; ++j) {
                if (base + j < a.count) {
                    float f[VEC];
                    G::template widen<VEC>(raw[j], f);
                    add_rows<VEC>(sum, f);
                }
            }
        }
    }
    if (a.out_bf16) store_bf16<VEC>(static_cast<uint16_t *>(a.out) + first, sum);
    else store_state<VEC>(static_cast<float *>(a.out) + first, sum);
}

template <typename G, int VEC, int DEPTH, int TREE>
__global__ void __launch_bounds__(kBlockThreads, tree_resident_blocks(TREE))
star_group_reduce_kernel(const __grid_constant__ ReduceArgs a)
{
    const int64_t n_vec = (a.n - a.head) / VEC;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kBlockThreads;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kBlockThreads + threadIdx.x; i < n_vec; i += stride)
        reduce_vector<G, VEC, DEPTH, TREE>(a, a.head + i * VEC);
    if constexpr (VEC > 1) {
        const int64_t e = edge_element<VEC>(a.n, a.head, n_vec);
        if (e >= 0) reduce_vector<G, 1, DEPTH, TREE>(a, e);
    }
}

// One or two sources (a parent without children, or with one: the common case
// when few workers are removed): a thread would have only one or two loads in
// flight, too few to cover the memory latency at any occupancy, so each thread
// takes two vectors per pass and issues the loads of both before it adds.
template <typename G, int VEC>
__global__ void __launch_bounds__(kBlockThreads, kResidentBlocks)
star_group_reduce_pair_kernel(const __grid_constant__ ReduceArgs a)
{
    constexpr int GB = VEC * G::kBytes;
    const int64_t n_vec = (a.n - a.head) / VEC;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kBlockThreads;
    const bool two_sources = a.count > 1;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kBlockThreads + threadIdx.x; i < n_vec; i += 2 * stride) {
        const int64_t first[2] = {a.head + i * VEC, a.head + (i + stride) * VEC};
        const bool second = i + stride < n_vec;
        Raw<GB> raw[2][2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (u == 0 || second) {
                raw[u][0] = load_stream<GB>(static_cast<const char *>(a.src[0]) + first[u] * G::kBytes);
                if (two_sources) raw[u][1] = load_stream<GB>(static_cast<const char *>(a.src[1]) + first[u] * G::kBytes);
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (u == 0 || second) {
                float sum[VEC];
                G::template widen<VEC>(raw[u][0], sum);
                if (two_sources) {
                    float f[VEC];
                    G::template widen<VEC>(raw[u][1], f);
                    add_rows<VEC>(sum, f);
                }
                if (a.out_bf16) store_bf16<VEC>(static_cast<uint16_t *>(a.out) + first[u], sum);
                else store_state<VEC>(static_cast<float *>(a.out) + first[u], sum);
            }
        }
    }
    const int64_t e = edge_element<VEC>(a.n, a.head, n_vec);
    if (e >= 0) reduce_vector<G, 1, 4, 0>(a, e);
}

// ---------------------------------------------------------------------------
// Tensor list.  The device workspace holds, in this order (each array 256-byte
// aligned): per-tensor TensorEntry records, the gradient pointer table
// [n_tensors * W], the snapshot pointer table [n_tensors * n_snapshot_sets] and
// tile_tensor[n_tiles] (tile -> tensor index).  Tiles of a tensor are
// consecutive; TensorEntry::first_tile is the tensor's first tile.  A tensor with
// `head` > 0 spends its first tile on those leading elements.
// ---------------------------------------------------------------------------
struct TensorEntry {
    float *params;
    float *momentum;
    int64_t size;          // elements
    int64_t first_tile;
    int32_t vec;           // elements per thread the tensor's buffer alignment allows (full width or 1)
    int32_t head;          // leading elements in front of the vector-aligned body (< vec)
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

// Extended tensor-list round: snapshots[t * n_sets + set] receives tensor t's
// parameters after the group that closes on a slot with snapshot_set[slot] ==
// set (-1: no snapshot for that group).
struct MultiExArgs {
    MultiArgs base;
    void *const *snapshots;         // [n_tensors * n_sets], entries may be null
    int32_t n_sets;
    int32_t snapshot_bf16;
    int8_t snapshot_set[kMaxWorkers];
};

struct NoMultiSnapshot {
    __device__ __forceinline__ NoSnapshot for_tensor(int32_t) const { return NoSnapshot(); }
};

struct StoreMultiSnapshot {
    const MultiExArgs *a;
    int32_t t;                         // the tensor: its row of the snapshot table is looked up at store time
    template <int VEC> __device__ __forceinline__ void operator()(int slot, int64_t first, const float (&p)[VEC]) const
    {
        const int set = a->snapshot_set[slot];
        if (set < 0) return;
        const unsigned long long *row =
            reinterpret_cast<const unsigned long long *>(a->snapshots) + static_cast<int64_t>(t) * a->n_sets;
        void *dst = reinterpret_cast<void *>(__ldg(row + set));
        if (dst == nullptr) return;
        if (a->snapshot_bf16) store_bf16<VEC>(static_cast<uint16_t *>(dst) + first, p);
        else store_state<VEC>(static_cast<float *>(dst) + first, p);
    }
};

struct MultiSnapshotSource {
    const MultiExArgs *a;
    __device__ __forceinline__ StoreMultiSnapshot for_tensor(int32_t t) const { return StoreMultiSnapshot{a, t}; }
};

// Element-by-element path for the ragged ends of a tensor and for tensors whose
// buffers do not share a vector alignment.  Kept out of line: it is cold, and
// inlining it next to the vector path costs registers there.
// Handles elements first, first + step, ... below end.
template <typename G, int DEPTH, int TREE, typename After>
__device__ __noinline__ void update_elements(const TensorEntry &te, const unsigned long long *row,
                                             int64_t first, int64_t end, int64_t step,
                                             const FlatSchedule &s, const Hyper &h, After after)
{
    auto grad_ptr = [&](int slot) -> const void * {
        return reinterpret_cast<const void *>(__ldg(row + s.member[slot]));
    };
    auto state_ptr = [&](int which) -> float * { return which == 0 ? te.params : te.momentum; };
    for (int64_t i = first; i < end; i += step)
        update_vector<G, 1, DEPTH, TREE>(state_ptr, i, s, h, grad_ptr, after);
}

// One block per tile of kBlockThreads * VEC elements (grid-stride over tiles);
// a thread owns one vector of its tile.
template <typename G, int VEC, int DEPTH, int TREE, typename Snapshots>
__device__ __forceinline__ void update_tiles(const MultiArgs &a, Snapshots snapshots)
{
    constexpr int64_t kTile = static_cast<int64_t>(kBlockThreads) * VEC;
    for (int64_t tile = blockIdx.x; tile < a.n_tiles; tile += gridDim.x) {
        const int32_t t = __ldg(a.tile_tensor + tile);
        const TensorEntry &te = a.tensors[t];
        const unsigned long long *row =
            reinterpret_cast<const unsigned long long *>(a.grads) + static_cast<int64_t>(t) * a.W;
        const int64_t size = te.size;
        const auto after = snapshots.for_tensor(t);
        // A vector-aligned tensor with leading elements spends its first tile on
        // them (through the element path); its later tiles cover the body.
        const int64_t local = tile - te.first_tile;
        const int64_t head = te.vec == VEC ? te.head : 0;
        if (te.vec == VEC && (head == 0 || local > 0)) {
            const int64_t i = head + (local - (head > 0 ? 1 : 0)) * kTile + static_cast<int64_t>(threadIdx.x) * VEC;
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
                update_vector<G, VEC, DEPTH, TREE>(state_ptr, i, a.sched, a.hyper, grad_ptr, after);
            } else if (i < size) {                   // the tensor's last, partial vector
                update_elements<G, DEPTH, TREE>(te, row, i, size, 1, a.sched, a.hyper, after);
            }
        } else {
            // The leading elements of an aligned tensor, or a tile of a tensor
            // whose buffers have no common vector alignment: element by element.
            // (A narrower vector path here was measured to cost the aligned path
            // a third of its bandwidth through register spills.)
            const int64_t begin = te.vec == VEC ? 0 : local * kTile;
            const int64_t end = te.vec == VEC ? head : min(size, begin + kTile);
            update_elements<G, DEPTH, TREE>(te, row, begin + threadIdx.x, end, kBlockThreads, a.sched, a.hyper, after);
        }
    }
}

template <typename G, int VEC, int DEPTH>
__global__ void __launch_bounds__(kBlockThreads, kResidentBlocks)
star_update_multi_kernel(const __grid_constant__ MultiArgs a)
{
    update_tiles<G, VEC, DEPTH, 0>(a, NoMultiSnapshot());
}

template <typename G, int VEC, int DEPTH, int TREE>
__global__ void __launch_bounds__(kBlockThreads, tree_resident_blocks(TREE))
star_update_multi_ex_kernel(const __grid_constant__ MultiExArgs a)
{
    update_tiles<G, VEC, DEPTH, TREE>(a.base, MultiSnapshotSource{&a});
}

}  // namespace star
