// Pieces shared by the per-instance-loss kernels: the running (max, sum) state of a one-pass
// log-sum-exp in base 2, its merge, and the label checks (Sec. "Asynchronous joint learning with CPU/GPU": the loss f of each batch instance).
#pragma once

#include <math.h>

#include "aa_internal.cuh"

namespace aa {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct LossParams {
    const void* logits;
    int64_t rows, cols, row_stride;
    const int32_t* labels;
    const int32_t* count_dev;
    const int32_t* row_idx;   // nullable: evaluated row k is stored row row_idx[k]; labels go by stored row
    int64_t n_stored;         // stored rows (bounds the list entries)
    float* out;
    Control* ctl;
};

struct RunState {
    float m;   // running maximum of t = x*log2(e)
    float s;   // sum of 2^(t - m)
};

__device__ __forceinline__ void absorb(RunState& st, const float* t, int n) {
    float vmax = t[0];
    for (int e = 1; e < n; ++e) vmax = fmaxf(vmax, t[e]);
    if (vmax > st.m) {
        st.s *= ex2_approx(st.m - vmax);   // st.m = -inf gives 0 * 0
        st.m = vmax;
    }
    const float ref = st.m == -INFINITY ? 0.0f : st.m;   // all -inf so far: every term is 2^-inf = 0
    for (int e = 0; e < n; ++e) st.s += ex2_approx(t[e] - ref);
}

// One vector of raw logits.  The maximum is taken on the logits themselves (scaling by log2(e) > 0
// keeps the order) and the scaling is fused with the shift:  2^(x log2(e) - ref)  is one FMA and
// one ex2 per element; two partial sums keep the additions from forming one chain.
template <int N>
__device__ __forceinline__ void absorb_vec(RunState& st, const float (&x)[N]) {
    float xmax = x[0];
#pragma unroll
    for (int e = 1; e < N; ++e) xmax = fmaxf(xmax, x[e]);
    const float vmax = xmax * kLog2e;
    if (vmax > st.m) {
        st.s *= ex2_approx(st.m - vmax);   // st.m = -inf gives 0 * 0
        st.m = vmax;
    }
    const float neg_ref = st.m == -INFINITY ? 0.0f : -st.m;   // all -inf so far: every term is 2^-inf = 0
    float a0 = 0.0f, a1 = 0.0f;
#pragma unroll
    for (int e = 0; e < N; e += 2) {
        a0 += ex2_approx(fmaf(x[e], kLog2e, neg_ref));
        if (e + 1 < N) a1 += ex2_approx(fmaf(x[e + 1], kLog2e, neg_ref));
    }
    st.s += a0 + a1;
}

// K vectors at once: one maximum, one comparison with the running maximum and one reference for all of them (the
// per-vector bookkeeping is a quarter of the instructions of a bf16 vector).
template <int K, int N>
__device__ __forceinline__ void absorb_vecs(RunState& st, const float (&x)[K][N]) {
    float xmax = x[0][0];
#pragma unroll
    for (int k = 0; k < K; ++k)
#pragma unroll
        for (int e = 0; e < N; ++e) xmax = fmaxf(xmax, x[k][e]);
    const float vmax = xmax * kLog2e;
    if (vmax > st.m) {
        st.s *= ex2_approx(st.m - vmax);   // st.m = -inf gives 0 * 0
        st.m = vmax;
    }
    const float neg_ref = st.m == -INFINITY ? 0.0f : -st.m;
    float a0 = 0.0f, a1 = 0.0f;
#pragma unroll
    for (int k = 0; k < K; ++k)
#pragma unroll
        for (int e = 0; e < N; e += 2) {
            a0 += ex2_approx(fmaf(x[k][e], kLog2e, neg_ref));
            a1 += ex2_approx(fmaf(x[k][e + 1], kLog2e, neg_ref));
        }
    st.s += a0 + a1;
}

__device__ __forceinline__ RunState merge(const RunState& a, const RunState& b) {
    RunState o;
    o.m = fmaxf(a.m, b.m);
    const float ref = o.m == -INFINITY ? 0.0f : o.m;
    o.s = a.s * ex2_approx(a.m - ref) + b.s * ex2_approx(b.m - ref);
    return o;
}

template <int WIDTH>
__device__ __forceinline__ RunState group_merge(RunState st) {
#pragma unroll
    for (int o = WIDTH / 2; o > 0; o >>= 1) {
        RunState other;
        other.m = __shfl_xor_sync(0xFFFFFFFFu, st.m, o);
        other.s = __shfl_xor_sync(0xFFFFFFFFu, st.s, o);
        st = merge(st, other);
    }
    return st;
}

__device__ __forceinline__ float finish_row(const RunState& st, float label_logit) {
    return (st.m + lg2_approx(st.s)) * kLn2 - label_logit;
}

__device__ __forceinline__ int64_t effective_rows(const LossParams& p) {
    int64_t rows = p.rows;
    if (p.count_dev) {
        const int64_t c = *p.count_dev;
        rows = c < 0 ? 0 : (c < rows ? c : rows);
    }
    return rows;
}

// Stored row of evaluated row k: k itself, or the list entry (outside the stored rows: -1, latches AA_ERR_BAD_INDEX).
__device__ __forceinline__ int64_t source_row(const LossParams& p, int64_t k) {
    if (!p.row_idx) return k;
    const int64_t r = __ldg(p.row_idx + k);
    if ((unsigned long long)r >= (unsigned long long)p.n_stored) {
        latch(p.ctl, AA_ERR_BAD_INDEX);
        return -1;
    }
    return r;
}

// Label of row r: >= 0 valid; -1 padding or invalid (invalid latches AA_ERR_BAD_INDEX).
__device__ __forceinline__ int checked_label(const LossParams& p, int64_t r) {
    const int y = __ldg(p.labels + r);
    if (y < 0) return -1;
    if (y >= p.cols) {
        latch(p.ctl, AA_ERR_BAD_INDEX);
        return -1;
    }
    return y;
}

}  // namespace aa
