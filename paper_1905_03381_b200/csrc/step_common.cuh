// Declarations shared by the Assistant-step kernels (labels + one SGD step of the linear
// Assistant; Sec. "Learning to generate smart training batches" label rule and objective, Algorithm 2: gradient, update).
#pragma once

#include "aa_internal.cuh"

namespace aa {

constexpr int kStepThreads = 512;
constexpr int kStepWarps = kStepThreads / 32;

struct StepParams {
    DenseFeat f;
    CsrFeat csr;
    const int32_t* row_idx;
    int64_t n_stored;
    int64_t m_host;
    const int32_t* count_dev;
    const float* loss;
    const float* score;   // optional: pre-activation of every STORED row under the current parameters (nullptr: recomputed)
    int thresh_mode;
    float threshold;
    float lr;
    float* w;
    float* b;
    float* partials;      // [parts][d_pad] column sums, then [parts] bias sums
    float* residual;      // per batch row (CSR path)
    int64_t d_pad;
    int rows_per_block;
    double* loss_sums;    // per-CTA shares of the batch loss sum (matrix-instruction kernel)
    AdamArgs adam;
    Control* ctl;
};

__device__ __forceinline__ int64_t batch_size(const StepParams& p) {
    int64_t m = p.m_host;
    if (p.count_dev) {
        const int64_t c = *p.count_dev;
        m = c < 0 ? 0 : (c < m ? c : m);
    }
    return m;
}

// Shrinking threshold T: the caller's value, or the mean of the batch losses.  Every CTA adds the
// losses in the same order (fp64), so all CTAs agree on T bit for bit.
__device__ __forceinline__ double block_threshold(const StepParams& p, int64_t m, double* red /* [warps] */) {
    if (p.thresh_mode == AA_THRESH_VALUE) return (double)p.threshold;
    double acc = 0.0;
    for (int64_t i = threadIdx.x; i < m; i += blockDim.x) acc += (double)__ldg(p.loss + i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    if (lane == 0) red[warp] = acc;
    __syncthreads();
    double total = 0.0;
    for (int wi = 0; wi < nwarps; ++wi) total += red[wi];
    __syncthreads();
    return m > 0 ? total / (double)m : 0.0;
}

__device__ __forceinline__ long long batch_row(const StepParams& p, int64_t i) {
    if (!p.row_idx) return i;
    const long long r = p.row_idx[i];
    if ((unsigned long long)r >= (unsigned long long)p.n_stored) {
        latch(p.ctl, AA_ERR_BAD_INDEX);
        return -1;
    }
    return r;
}


// Adds the per-CTA partial sums in CTA order and applies  w <- w - lr * grad  (defined in assistant_step.cu).
aa_status launch_linear_apply(aa_ctx_impl* c, const StepParams& p, int parts);
// Matrix-instruction variant for aligned bf16 rows of 256..3072 features (a multiple of 16); AA_ERR_UNSUPPORTED otherwise.
// *parts_out = 0 when the kernel has taken the update itself (no apply launch needed).
aa_status launch_assistant_grad_dense_mma(aa_ctx_impl* c, StepParams& p, int* parts_out);
// Variant for callers that pass the screening scores (p.score): same shapes as the matrix-instruction variant, no dot products.
aa_status launch_assistant_grad_dense_scored(aa_ctx_impl* c, StepParams& p, int* parts_out);
// Bulk-copy variant of the dense gradient kernel; AA_ERR_UNSUPPORTED when the shape does not fit its ring.
aa_status launch_assistant_grad_dense_tma(aa_ctx_impl* c, StepParams& p, int* parts_out);

}  // namespace aa
