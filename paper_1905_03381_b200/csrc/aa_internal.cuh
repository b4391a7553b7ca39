// Internal declarations shared by the kernels of the AutoAssist batch-generator library.
// Nothing here is part of the C ABI (that is include/autoassist.h).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "autoassist.h"

namespace aa {

// Device-resident control block at the start of the caller's workspace.
struct Control {
    unsigned int ticket;   // next tile to hand out (dynamic tile order = look-back order)
    unsigned int done;     // CTAs of the running scan kernel that have finished
    unsigned int epoch;    // generation of the look-back flags; bumped by the last CTA of each scan
    int status;            // first device-side condition latched (aa_status), 0 = none
    unsigned int pad0[28];
    // second 128-byte line: the counters the gradient kernel's CTAs poll, kept away from the ticket counter that the
    // same kernel's producers hammer with atomics
    unsigned int sums_in;  // CTAs of the running gradient kernel that have published their share of the loss sum
    unsigned int grad_done;  // CTAs of the running gradient kernel that have written their partial sums
    unsigned int applied;  // CTAs of the running gradient kernel that have seen every CTA's partial sums
    unsigned int pad1[29];
};
static_assert(sizeof(Control) == 256, "control block is one 256-byte line group");

constexpr int kMaxTileRows = 1024;     // rows of one compaction tile (multiple of 32)
constexpr int kScanThreads = 128;      // CTA size of the score/shrink/compact kernels
constexpr int kMaxParts = 1024;        // upper bound on per-CTA gradient partials
constexpr unsigned kSpinLimit = 1u << 22;   // polls before a look-back wait gives up

// Optimizer of the Assistant update: plain SGD, or Adam with caller-owned moment arrays laid out like the
// flattened parameters (linear: w[d] then b; two-layer: W1[hidden*d], b1[hidden], w2[hidden], b2).
struct AdamArgs {
    int on;
    float beta1, beta2, eps;
    float corr1, corr2;      // 1 / (1 - beta1^t), 1 / (1 - beta2^t) for this step
    float* m;
    float* v;
};

struct aa_ctx_impl {
    char* ws;
    size_t ws_bytes;
    cudaStream_t stream;
    int device;
    int sm_count;
    int64_t max_rows, max_d, max_hidden;
    Control* ctl;
    unsigned long long* tile_state;   // one packed (flag, value) word per tile
    int64_t max_tiles;
    float* row_scratch;               // max_rows floats: row losses / residuals
    float* partials;                  // gradient partial sums
    int64_t partial_floats;
    AdamArgs adam;                    // optimizer of the step being enqueued (on = 0: SGD)
    const float* step_score;          // pre-activations handed to the step being enqueued (nullptr: recomputed)
    int64_t launches;
    uint64_t scans_since_clear;
    // two-layer Assistant step (present when the context was sized with max_hidden > 0)
    void* mlp_pt;                     // gate bits and residual terms of the batch, then the gate bits of the last screened pool
    // the gates [a > 0] that the last two-layer screening on this context left behind (32 bytes per candidate), and what
    // they belong to: a later update on that pool's rows under unchanged parameters may use them instead of a forward pass
    uint32_t* mlp_gate_cand;
    const void* gate_feat;            // feature base pointer of that pool (nullptr: nothing usable)
    const void* gate_w1;              // the bf16 first-layer weights it was screened with
    int64_t gate_n;                   // its stored rows
    float* mlp_small;                 // per-CTA column-sum partials
    float* mlp_part;                  // split-K partials of the W1 gradient
    size_t mlp_part_bytes;
};

// Arguments of the shrink + compaction tail shared by every scoring front end.
struct ShrinkParams {
    Control* ctl;
    unsigned long long* tile_state;
    int64_t n_cand;          // candidates in the pool
    int64_t n_stored;        // stored rows (bound for row_idx entries)
    const int32_t* row_idx;  // optional candidate list
    int64_t id_base;
    float mix;               // gamma of Algorithm 1
    int hard;                // 1: keep iff value >= hard_threshold (hard shrinking, no random draw)
    float hard_threshold;
    uint32_t seed_lo, seed_hi, step_lo, step_hi;
    int32_t* out_idx;
    int64_t capacity;
    int32_t* out_count;
    float* out_score;
    uint8_t* out_mask;
    int tile_rows;
    unsigned int n_tiles;
};

// ---------------------------------------------------------------- device helpers
#ifdef __CUDACC__

// One parameter's update from its mean gradient `grad` (Algorithm 2: Assistant.update).  SGD: param - lr * grad.
// Adam (the optimizer the paper trained the Assistant with, Sec. "Image classification"): biased moments in a.m / a.v, bias-corrected step.
__device__ __forceinline__ float adam_update(const AdamArgs& a, float param, float grad, float lr, int64_t j) {
    const float m = a.beta1 * a.m[j] + (1.0f - a.beta1) * grad;
    const float v = a.beta2 * a.v[j] + (1.0f - a.beta2) * grad * grad;
    a.m[j] = m;
    a.v[j] = v;
    return param - lr * (m * a.corr1) / (sqrtf(v * a.corr2) + a.eps);
}

__device__ __forceinline__ void latch(Control* ctl, int code) { atomicCAS(&ctl->status, 0, code); }

// Programmatic dependent launch: wait for every earlier kernel of the stream to have finished (and its writes to be
// visible); a no-op for a kernel launched in plain stream order.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel of the stream (if it was launched with programmatic serialisation) take SM resources as they
// free up; it still waits in grid_dependency_wait() until this kernel has finished.
__device__ __forceinline__ void grid_dependency_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float lg2_approx(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// g = sigmoid(s) without overflow on either side.
__device__ __forceinline__ float sigmoid_f32(float s) {
    float e = expf(-fabsf(s));
    float pos = 1.0f / (1.0f + e);
    return s >= 0.0f ? pos : e * pos;
}

// Philox4x32-10 (Salmon et al., SC'11); returns output word 0 only.
__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                         uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c0;
}

// The uniform draw c of Algorithm 1 for instance `id` at `step`: 24 random bits scaled to [0, 1).
__device__ __forceinline__ float philox_uniform(const ShrinkParams& p, uint64_t id) {
    const uint32_t w = philox4x32_10_word0((uint32_t)id, (uint32_t)(id >> 32), p.step_lo, p.step_hi, p.seed_lo, p.seed_hi);
    return (float)(w >> 8) * (1.0f / 16777216.0f);
}

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

__device__ __forceinline__ float bf16_lo(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t packed) { return __uint_as_float(packed & 0xFFFF0000u); }

// 16-byte vector of stored elements widened to fp32.
template <typename T>
struct Vec;
template <>
struct Vec<float> {
    static constexpr int kElems = 4;
    __device__ static __forceinline__ void unpack(const uint4& v, float (&out)[4]) {
        out[0] = __uint_as_float(v.x); out[1] = __uint_as_float(v.y);
        out[2] = __uint_as_float(v.z); out[3] = __uint_as_float(v.w);
    }
    __device__ static __forceinline__ void load(const float* p, float (&out)[4]) {
        unpack(__ldg(reinterpret_cast<const uint4*>(p)), out);
    }
    __device__ static __forceinline__ float one(const float* p) { return __ldg(p); }
    // weights staged in shared memory: plain order, lane v reads one float4 (conflict-free)
    __device__ static __forceinline__ int w_index(int j, int /*nvec*/) { return j; }
    __device__ static __forceinline__ void load_w(const float* w_s, int /*nvec*/, int v, float (&out)[4]) {
        const float4 a = reinterpret_cast<const float4*>(w_s)[v];
        out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
    }
};
template <>
struct Vec<uint16_t> {   // bf16 bit patterns
    static constexpr int kElems = 8;
    __device__ static __forceinline__ void unpack(const uint4& v, float (&out)[8]) {
        out[0] = bf16_lo(v.x); out[1] = bf16_hi(v.x);
        out[2] = bf16_lo(v.y); out[3] = bf16_hi(v.y);
        out[4] = bf16_lo(v.z); out[5] = bf16_hi(v.z);
        out[6] = bf16_lo(v.w); out[7] = bf16_hi(v.w);
    }
    __device__ static __forceinline__ void load(const uint16_t* p, float (&out)[8]) {
        unpack(__ldg(reinterpret_cast<const uint4*>(p)), out);
    }
    __device__ static __forceinline__ float one(const uint16_t* p) { return __uint_as_float((uint32_t)__ldg(p) << 16); }
    // weights staged in shared memory: the 8 weights of vector v are split into two float4
    // planes so that consecutive lanes read consecutive 16-byte words (conflict-free)
    __device__ static __forceinline__ int w_index(int j, int nvec) {
        const int v = j >> 3, e = j & 7;
        return (e >> 2) * nvec * 4 + v * 4 + (e & 3);
    }
    __device__ static __forceinline__ void load_w(const float* w_s, int nvec, int v, float (&out)[8]) {
        const float4 a = reinterpret_cast<const float4*>(w_s)[v];
        const float4 b = reinterpret_cast<const float4*>(w_s)[nvec + v];
        out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
        out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
    }
};

#endif  // __CUDACC__

// ---------------------------------------------------------------- host-side launchers (one per .cu)
struct DenseFeat {
    const void* base;
    int dtype;
    int64_t d, row_stride;
    const float* w;
    const float* b;
};
struct CsrFeat {
    const int32_t* indptr;
    const int32_t* col;
    const float* val;
    int64_t d;
    const float* w;
    const float* b;
    float mean_nnz;
};

// Two-layer Assistant on dense bf16 rows: W1_bf16 is [hidden x d] row-major.
struct MlpFeat {
    const void* x;
    int64_t n, d, row_stride;
    const void* W1_bf16;
    const float* b1;
    const float* w2;
    const float* b2;
    int64_t hidden;
};
// tcgen05 scoring kernel (aligned bf16 rows, hidden a multiple of 16 up to 256, no candidate list).
aa_status launch_score_shrink_mlp(aa_ctx_impl* c, const MlpFeat& f, ShrinkParams sp);

// Labels + one SGD step of the two-layer Assistant on the batch rows (updates W1_master, W1_bf16, b1, w2, b2).
aa_status launch_assistant_step_mlp(aa_ctx_impl* c, const MlpFeat& f, float* W1_master, const int32_t* row_idx, int64_t n_stored,
                                    int64_t m_host, const int32_t* count_dev, const float* loss, float lr, int thresh_mode,
                                    float threshold);
// Workspace of that step: returns the bytes of the split-K partials, sets the bytes of the batch hand-over + pool gate
// bits (`pt_bytes`, the pool's gate bits start at *gate_off inside it) and of the small partials.
size_t mlp_step_workspace_bytes(int64_t max_rows, int64_t max_d, int64_t max_hidden, size_t* pt_bytes, size_t* small_bytes,
                                size_t* gate_off);

aa_status launch_score_shrink_dense(aa_ctx_impl* c, const DenseFeat& f, ShrinkParams sp);
// Bulk-copy (cp.async.bulk + mbarrier) variant for 16-byte aligned rows; AA_ERR_UNSUPPORTED when
// the shape does not fit its shared-memory ring, in which case the caller uses the load-based kernel.
aa_status launch_score_shrink_dense_tma(aa_ctx_impl* c, const DenseFeat& f, ShrinkParams sp);
// Tile geometry + scan state of a shrink launch (sets tile_rows, n_tiles, ctl, tile_state).
aa_status finish_shrink_params(aa_ctx_impl* c, ShrinkParams& sp, int tile_rows);
aa_status launch_score_shrink_csr(aa_ctx_impl* c, const CsrFeat& f, ShrinkParams sp);
aa_status launch_shrink_from_scores(aa_ctx_impl* c, const float* score, ShrinkParams sp);

// Bulk-copy variant for 16-byte aligned rows (writes p.out); AA_ERR_UNSUPPORTED when the shape does not fit.
struct LossParams;

aa_status launch_batch_cut(aa_ctx_impl* c, const int32_t* idx, const int32_t* count_dev, int64_t m_host, int64_t n_cand,
                           int64_t n_stored, int64_t batch_size, const int32_t* lengths, int64_t token_budget, int32_t* out_m,
                           int32_t* out_consumed, int32_t* out_offsets, int64_t offsets_capacity);

aa_status launch_instance_loss(aa_ctx_impl* c, const aa_logits& lg, const int32_t* labels, const int32_t* offsets,
                               int64_t n_seg, const int32_t* count_dev, float* out_loss, const int32_t* row_idx = nullptr,
                               int64_t n_rows = 0);

aa_status launch_assistant_step_dense(aa_ctx_impl* c, const DenseFeat& f, const int32_t* row_idx, int64_t n_stored,
                                      int64_t m_host, const int32_t* count_dev, const float* loss, float* w, float* b,
                                      float lr, int thresh_mode, float threshold);
aa_status launch_assistant_step_csr(aa_ctx_impl* c, const CsrFeat& f, const int32_t* row_idx, int64_t n_stored,
                                    int64_t m_host, const int32_t* count_dev, const float* loss, float* w, float* b,
                                    float lr, int thresh_mode, float threshold);

// Launch on the context's stream with programmatic stream serialisation: the kernel's CTAs may be placed on SMs while
// the previous kernel of the stream is still draining (its launch latency and prologue then overlap that kernel's
// tail).  Such a kernel MUST call grid_dependency_wait() before it reads or writes anything an earlier kernel of the
// stream may have written; kernels that precede it call grid_dependency_release() once their own CTAs are all placed.
// cooperative = the CTAs wait for one another (the grid must be resident at once).
cudaError_t launch_overlapped(aa_ctx_impl* c, const void* kernel, dim3 grid, dim3 block, void** args, size_t smem, bool cooperative);

// Convolution + rectifier + average pooling of every stored image row (the convolutional Assistant's feature map).
aa_status launch_conv_pool_features(aa_ctx_impl* c, const void* x, int dtype, int64_t n, int64_t row_stride, const aa_conv& cv,
                                    float* phi, int64_t phi_stride);

// Persistent-grid size for a kernel: CTAs that fit on the device at once.
int resident_ctas(aa_ctx_impl* c, const void* kernel, int threads, size_t dyn_smem);

inline aa_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? AA_OK : AA_ERR_CUDA; }

}  // namespace aa
