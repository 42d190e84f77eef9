/*
 * CPU oracle for STAR's parameter-server-side grouped aggregation + update.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, serial, obviously-correct
 * statement of what the grouped update computes.  It is compiled with gcc,
 * called from the test-suite, the smoke check and the CPU-baseline leg of the
 * benchmark, and from nowhere else.  It shares no code, header, table or
 * helper with the CUDA library and neither side includes the other.
 *
 * What it follows (paper: "Straggler Tolerant and Resilient DL Training on
 * Homogeneous GPUs"):
 *   - Section I:    SSGD updates parameters only once gradients from all N
 *                   workers are in; ASGD updates on the gradient of any one
 *                   worker.
 *   - Section I, contribution (2) and Section IV-B: the static x-order mode
 *                   uses the gradients of x workers for each parameter update;
 *                   the dynamic x-order mode uses the gradient reports of one
 *                   worker cluster for each update.
 *   - Section IV-C1 (text before Eq. 2): clusters are taken in ascending
 *                   order of their largest iteration time, i.e. the groups of
 *                   a round are ORDERED and are applied one after another.
 *   - Section II:   the PS updates the parameters (one master copy).
 *
 * The paper never prints the update rule.  The reading used here: every group
 * update is one complete SGD step with momentum (dampening 0, no Nesterov)
 * and L2 weight decay folded into the gradient, on the MEAN of the group's
 * gradients:
 *
 *     for k = 0 .. K-1 (schedule order):
 *         s    = g[m_k0][i] + g[m_k1][i] + ...      (left to right, CSR order)
 *         gbar = s / |G_k|
 *         d    = gbar + wd * p[i]
 *         v[i] = mu * v[i] + d
 *         p[i] = p[i] - lr * v[i]
 *
 * In-group summation order (sum_order argument):
 *   0  linear: left to right in the listed member order (the default reading).
 *   1  tree:   pairwise, as gradients are combined along a binary aggregation
 *              tree (Section IV-D2b, workers add their children's gradients to
 *              their own on the way up): tree(m_0..m_{c-1}) = the member itself
 *              for c = 1, otherwise tree(first h) + tree(remaining c - h) with
 *              h the largest power of two below c.
 *
 * Two variants:
 *   oracle_group_update_f32  canonical binary32 sequence; each line above is
 *                            ONE correctly rounded IEEE operation: fp32 add,
 *                            fp32 true division, and three fused multiply-adds
 *                            d=fma(wd,p,gbar), v=fma(mu,v,d), p=fma(-lr,v,p).
 *   oracle_group_update_f64  the same loop in binary64 without fused
 *                            operations: the shadow that says how far the
 *                            fp32 sequence is from the real-number result.
 *
 * Pins (tests/test_oracle_pins.py): hand-worked dyadic example, exact-rational
 * brute force, closed forms (mu=wd=0; wd=0; 2x2 affine recurrence), the
 * library SGD optimizer of PyTorch in fp64, SSGD == one mean update, fused K
 * groups == K single-group calls, member-permutation invariance.
 *
 * All-reduce architecture (Section IV-B, paragraph "All-reduce architecture";
 * Section IV-C1, Eq. 3).  x stragglers leave the ring and report to a parent
 * each; a parent adds the gradients of its children (those that reported
 * before it stopped waiting) to its own and hands the aggregate to the ring;
 * the ring sums the aggregates of its members; the update uses the gradients
 * of N - x + q workers.  Two functions state the arithmetic of that round:
 *   oracle_group_reduce_f32        what a parent forwards: the binary32 sum of
 *                                  the listed buffers (own gradient first,
 *                                  then the children), left to right or
 *                                  pairwise, stored as binary32 or rounded to
 *                                  bf16.
 *   oracle_update_from_sums_f32    one update from R partial sums: they are
 *                                  added left to right in the listed (ring)
 *                                  order, the mean divides by the number of
 *                                  gradient reports behind them (N - x + q,
 *                                  the batch Eq. 3 counts), then the three
 *                                  fused multiply-adds of a group update.
 * The paper fixes neither order; oracle/all_reduce.py composes the two into a
 * round and states the reading.  Pins: tests/test_all_reduce_oracle.py.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

enum { ORACLE_DTYPE_F32 = 0, ORACLE_DTYPE_BF16 = 1 };

/* bf16 is the upper half of a binary32: widening is exact. */
static float widen_bf16(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* binary32 -> bf16, round to nearest, ties to even; NaN stays NaN (quiet). */
static uint16_t narrow_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u)
        return (uint16_t)((u >> 16) | 0x0040u);
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

static float grad_at(const void *buf, int dtype, int64_t i)
{
    if (dtype == ORACLE_DTYPE_BF16)
        return widen_bf16(((const uint16_t *)buf)[i]);
    return ((const float *)buf)[i];
}

/* Pairwise (tree) sum of members[0..count) at element i, binary32. */
static float tree_sum_f32(const void *const *grads, int dtype, const int32_t *members, int count, int64_t i)
{
    if (count == 1)
        return grad_at(grads[members[0]], dtype, i);
    int h = 1;
    while (2 * h < count)
        h *= 2;
    return tree_sum_f32(grads, dtype, members, h, i) + tree_sum_f32(grads, dtype, members + h, count - h, i);
}

static double tree_sum_f64(const void *const *grads, int dtype, const int32_t *members, int count, int64_t i)
{
    if (count == 1)
        return (double)grad_at(grads[members[0]], dtype, i);
    int h = 1;
    while (2 * h < count)
        h *= 2;
    return tree_sum_f64(grads, dtype, members, h, i) + tree_sum_f64(grads, dtype, members + h, count - h, i);
}

/* 1 if the schedule is one the definition covers, else 0.  The public
 * functions return 0 on success and 1 on such a schedule. */
static int schedule_ok(const int32_t *group_offsets, const int32_t *group_members,
                       int n_groups, int W)
{
    if (n_groups < 0 || W < 0)
        return 0;
    if (n_groups == 0)
        return 1;
    if (!group_offsets || !group_members || group_offsets[0] != 0)
        return 0;
    for (int k = 0; k < n_groups; ++k)
        if (group_offsets[k + 1] <= group_offsets[k])
            return 0; /* the mean of an empty group is undefined */
    for (int j = 0; j < group_offsets[n_groups]; ++j) {
        if (group_members[j] < 0 || group_members[j] >= W)
            return 0;
        for (int l = 0; l < j; ++l)
            if (group_members[l] == group_members[j])
                return 0; /* a gradient report feeds exactly one update */
    }
    return 1;
}

/*
 * Canonical binary32 oracle.  lrs has one learning rate per group (Section
 * IV-C1, "Scaling learning rate after switching": the rate follows the number
 * of gradient reports y used by the update); pass the same value K times for
 * a single rate.  snapshots is NULL, or K pointers of which the non-NULL ones
 * receive the parameters as they stand right after that group's update: the
 * copy the PS sends back to the workers of that group (Section II), as
 * binary32 (snapshot_dtype 0) or rounded to bf16 (snapshot_dtype 1).
 */
int oracle_group_update_f32(float *params, float *momentum,
                            const void *const *grads, int W, int grad_dtype,
                            int64_t n, const int32_t *group_offsets,
                            const int32_t *group_members, int n_groups,
                            const float *lrs, float mu, float wd,
                            void *const *snapshots, int snapshot_dtype, int sum_order)
{
    if (!schedule_ok(group_offsets, group_members, n_groups, W) || sum_order < 0 || sum_order > 1 ||
        snapshot_dtype < 0 || snapshot_dtype > 1)
        return 1;
    for (int64_t i = 0; i < n; ++i) {
        float p = params[i];
        float v = momentum[i];
        for (int k = 0; k < n_groups; ++k) {
            const int first = group_offsets[k];
            const int last = group_offsets[k + 1];
            float s;
            if (sum_order == 1) {
                s = tree_sum_f32(grads, grad_dtype, group_members + first, last - first, i);
            } else {
                s = grad_at(grads[group_members[first]], grad_dtype, i);
                for (int j = first + 1; j < last; ++j)
                    s = s + grad_at(grads[group_members[j]], grad_dtype, i);
            }
            const float gbar = s / (float)(last - first);
            const float d = fmaf(wd, p, gbar);
            v = fmaf(mu, v, d);
            p = fmaf(-lrs[k], v, p);
            if (snapshots && snapshots[k]) {
                if (snapshot_dtype == ORACLE_DTYPE_BF16)
                    ((uint16_t *)snapshots[k])[i] = narrow_bf16(p);
                else
                    ((float *)snapshots[k])[i] = p;
            }
        }
        params[i] = p;
        momentum[i] = v;
    }
    return 0;
}

/* Binary64 shadow: same order, plain multiply and add, no fused operation. */
int oracle_group_update_f64(double *params, double *momentum,
                            const void *const *grads, int W, int grad_dtype,
                            int64_t n, const int32_t *group_offsets,
                            const int32_t *group_members, int n_groups,
                            const double *lrs, double mu, double wd,
                            double *const *snapshots, int sum_order)
{
    if (!schedule_ok(group_offsets, group_members, n_groups, W) || sum_order < 0 || sum_order > 1)
        return 1;
    for (int64_t i = 0; i < n; ++i) {
        double p = params[i];
        double v = momentum[i];
        for (int k = 0; k < n_groups; ++k) {
            const int first = group_offsets[k];
            const int last = group_offsets[k + 1];
            double s;
            if (sum_order == 1) {
                s = tree_sum_f64(grads, grad_dtype, group_members + first, last - first, i);
            } else {
                s = (double)grad_at(grads[group_members[first]], grad_dtype, i);
                for (int j = first + 1; j < last; ++j)
                    s = s + (double)grad_at(grads[group_members[j]], grad_dtype, i);
            }
            const double gbar = s / (double)(last - first);
            const double d = gbar + wd * p;
            v = mu * v + d;
            p = p - lrs[k] * v;
            if (snapshots && snapshots[k])
                snapshots[k][i] = p;
        }
        params[i] = p;
        momentum[i] = v;
    }
    return 0;
}

/* 1 if members[0..count) are distinct workers in [0, W), count >= 1. */
static int members_ok(const int32_t *members, int count, int W)
{
    if (count < 1 || !members)
        return 0;
    for (int j = 0; j < count; ++j) {
        if (members[j] < 0 || members[j] >= W)
            return 0;
        for (int l = 0; l < j; ++l)
            if (members[l] == members[j])
                return 0;
    }
    return 1;
}

/*
 * Section IV-B, all-reduce architecture: a parent aggregates "the gradients
 * from its children and its own gradients".  out[i] = g[m_0][i] + g[m_1][i] +
 * ... in binary32, in the listed order (sum_order 0) or pairwise (sum_order
 * 1, as tree_sum_f32 above); out is binary32 (out_dtype 0) or the sum rounded
 * to bf16, nearest even (out_dtype 1).  Returns 0, or 1 for arguments outside
 * the definition.
 */
int oracle_group_reduce_f32(void *out, int out_dtype, const void *const *grads, int W, int grad_dtype,
                            int64_t n, const int32_t *members, int count, int sum_order)
{
    if (!members_ok(members, count, W) || sum_order < 0 || sum_order > 1 || out_dtype < 0 || out_dtype > 1)
        return 1;
    for (int64_t i = 0; i < n; ++i) {
        float s;
        if (sum_order == 1) {
            s = tree_sum_f32(grads, grad_dtype, members, count, i);
        } else {
            s = grad_at(grads[members[0]], grad_dtype, i);
            for (int j = 1; j < count; ++j)
                s = s + grad_at(grads[members[j]], grad_dtype, i);
        }
        if (out_dtype == ORACLE_DTYPE_BF16)
            ((uint16_t *)out)[i] = narrow_bf16(s);
        else
            ((float *)out)[i] = s;
    }
    return 0;
}

/*
 * Section IV-B / Eq. 3: the one update of an all-reduce round.  sums[0..R) are
 * the binary32 aggregates of the R ring members in ring order; n_reports is
 * the number of gradient reports they contain together (N - x + q >= R).
 *     s    = sums[0][i] + sums[1][i] + ...     left to right
 *     gbar = s / n_reports
 *     d = fma(wd, p, gbar) ; v = fma(mu, v, d) ; p = fma(-lr, v, p)
 */
int oracle_update_from_sums_f32(float *params, float *momentum, const float *const *sums, int R, int64_t n,
                                int n_reports, float lr, float mu, float wd)
{
    if (R < 1 || n_reports < R || !sums)
        return 1;
    for (int64_t i = 0; i < n; ++i) {
        float s = sums[0][i];
        for (int r = 1; r < R; ++r)
            s = s + sums[r][i];
        const float gbar = s / (float)n_reports;
        const float d = fmaf(wd, params[i], gbar);
        const float v = fmaf(mu, momentum[i], d);
        momentum[i] = v;
        params[i] = fmaf(-lr, v, params[i]);
    }
    return 0;
}
