// Labels + one SGD step of the two-layer Assistant g = sigmoid(w2 . relu(W1 x + b1) + b2)
// (Sec. "Learning to generate smart training batches" label rule and objective; Algorithm 2: Assistant.gradient, Assistant.update),
// back-propagated through both layers on the tcgen05 tensor cores.
//
//   mlp_residual_kernel  forward pass over the batch rows under the current parameters (same
//                        TMA/MMA pipeline as scoring, but in tiles of 128 rows whose two
//                        accumulators alternate: the passes over one tile's accumulator run
//                        while the products of the next tile are issued), then per row  z = 1[loss > T],
//                        r = sigmoid(s) - z,  and per hidden unit u the gate [a_iu > 0] of
//                        delta1_iu = r_i w2_u [a_iu > 0].  What leaves for the W1 gradient is small:
//                        the gates as one bit each (64 rows x 256 units per 2 KB block) and r_i as
//                        two bf16 terms r_hi + r_lo (16 mantissa bits together).  The column sums
//                        sum_i r_i relu(a_iu) (-> grad w2), sum_i r_i [a_iu > 0] (-> grad b1) and
//                        sum_i r_i (-> grad b2) stay in fp32 and leave as per-CTA partials.
//   mlp_w1_grad_kernel   G[u][k] = sum_i P[i][u] x_ik with P[i][u] = r_i [a_iu > 0]: a [hidden x rows] x
//                        [rows x d] contraction over the batch rows.  A CTA owns 256 feature columns and a
//                        slice of the rows (split-K).  Per 64-row slice the feature rows arrive by TMA as an
//                        MN-major operand (the contraction runs down the rows, 128-byte swizzle), while eight
//                        warps BUILD the other operand in shared memory from the gate bits and r: one
//                        K-major [hidden x 64] bf16 tile for r_hi and one for r_lo, both multiplied into the
//                        same two [128 x 256] fp32 accumulators in TMEM (hidden units 0..127 and 128..255).
//                        No P matrix crosses HBM or L2, and the bf16 rounding of r (2^-9) does not reach the
//                        gradient.  Partials go to the workspace.
//   mlp_apply_w1_kernel  W1 <- W1 - lr (w2_u / M) sum_splits G ; W1_bf16 <- round-to-nearest-even(W1).
//   mlp_apply_small_kernel  b1, w2, b2 from the column-sum partials (reads the old w2 first).
//
// When the caller passes the scores of the screening that produced the batch and that screening ran on this context
// (its gates [a > 0] are still in the workspace, one bit per candidate and unit), the forward pass is not repeated:
//   mlp_prepare_kernel   per batch row i (stored row rho_i):  r_i = sigmoid(score[rho_i]) - z_i, its two bf16 terms, the
//                        gate words of rho_i transposed into the block layout above, and the column sums
//                        sum_i r_i [a_iu > 0] and sum_i r_i.
// The W1 gradient runs as before.  grad w2 needs sum_i r_i relu(a_iu); with relu(a_iu) = [a_iu > 0] (W1b_u . x_i + b1_u) that is
//   sum_k W1b_uk G_uk + b1_u sum_i r_i [a_iu > 0],
// so mlp_apply_w1_kernel, which holds G and the old W1 anyway, also leaves the dot products sum_k W1b_uk G_uk (per warp,
// added in a fixed order by mlp_apply_small_kernel).
#include <cuda_bf16.h>
#include <math.h>

#include "mlp_pipeline.cuh"
#include "step_common.cuh"

namespace aa {

namespace {

constexpr int kStepMlpThreads = 576;          // warps 12..17 only help with row gathers
constexpr int kStepEpiWarps = 8;              // two sets of four: set b drains accumulator b
constexpr int kMaxMlpCtas = 192;              // bound on the grids below (workspace sizing)
constexpr int kFeatChunk = 256;               // feature columns per CTA of the W1-gradient kernel
constexpr int kRowSlice = 64;                 // batch rows per K-slice of the W1-gradient kernel

struct MlpStepParams {
    // batch
    const int32_t* row_idx;
    int64_t n_stored, m_host;
    const int32_t* count_dev;
    const float* loss;
    int thresh_mode;
    float threshold;
    float lr;
    // parameters
    float* W1;
    __nv_bfloat16* W1_bf16;
    float* b1;
    float* w2;
    float* b2;
    int64_t d;
    MlpGeom g;
    // workspace
    uint32_t* gate_bits;      // [pitch / 64][kMaxHidden][2]: bit (i & 31) of word (i >> 5) & 1 = [a_iu > 0] for row i, unit u
    __nv_bfloat16* r_hi;      // [pitch]: r_i rounded to bf16
    __nv_bfloat16* r_lo;      // [pitch]: r_i - r_hi rounded to bf16
    int64_t pitch;            // batch rows rounded up to whole tiles
    float* small;             // [ctas][2 * kMaxHidden + 1]: sum r relu(a), sum P, sum r
    float* part;              // [splits][hidden][d_pad]
    int64_t d_pad;
    int n_chunks, splits;
    // route that reuses the screening's scores and gates (all nullptr / 0 when the forward pass is recomputed)
    const float* score;           // pre-activation of every stored row
    const uint32_t* gate_cand;    // [stored rows][kMaxHidden / 32] gate words of every stored row
    float* gw2_part;              // [hidden][gw2_segs]: sum over 128 feature columns of W1b_uk G_uk
    int gw2_segs;
    AdamArgs adam;
    Control* ctl;
};

__device__ __forceinline__ int64_t mlp_batch_size(const MlpStepParams& p) {
    int64_t m = p.m_host;
    if (p.count_dev) {
        const int64_t c = *p.count_dev;
        m = c < 0 ? 0 : (c < m ? c : m);
    }
    return m;
}

// Sum over the warp's 32 lanes of each of 32 per-lane values: afterwards v[0] of lane l holds the
// total of element l (31 shuffles instead of 32 five-step reductions).
__device__ __forceinline__ float lanes_transpose_sum(float (&v)[32], int lane) {
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int j = 0; j < off; ++j) {
            const float send = upper ? v[j] : v[j + off];
            const float keep = upper ? v[j + off] : v[j];
            v[j] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, off);
        }
    }
    return v[0];
}

__device__ __forceinline__ void step_give_up(const MlpStepParams& p, TilePipe* tp) {
    latch(p.ctl, AA_ERR_SCAN_TIMEOUT);
    *(volatile int*)&tp->abort_flag = 1;
}

// ---------------------------------------------------------------- forward + residuals + P^T
template <bool GATHER>
__global__ void __launch_bounds__(kStepMlpThreads, 1)
mlp_residual_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, MlpStepParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    float* b1_s = reinterpret_cast<float*>(ring + (size_t)kHalfStages * p.g.stage_bytes);
    float* w2_s = b1_s + kMaxHidden;
    float* col_s = w2_s + kMaxHidden;                        // [kStepEpiWarps][2][kMaxHidden] column sums per warp
    double* red = reinterpret_cast<double*>(col_s + kStepEpiWarps * 2 * kMaxHidden);   // [warps]
    float* rsum_s = reinterpret_cast<float*>(red + kStepMlpThreads / 32);              // [kStepEpiWarps]
    TilePipe* tp = reinterpret_cast<TilePipe*>(rsum_s + kStepEpiWarps);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int hidden = p.g.hidden;
    if (tid == 0) {
        tile_pipe_init(tp, kStepEpiWarps / 2);
        mbar_fence_init();
        prefetch_tensormap(&map_x);
        prefetch_tensormap(&map_w);
    }
    for (int j = tid; j < kMaxHidden; j += kStepMlpThreads) {
        b1_s[j] = j < hidden ? p.b1[j] : 0.0f;
        w2_s[j] = j < hidden ? p.w2[j] : 0.0f;
    }
    if (warp == 2) tmem_alloc(&tp->tmem_base, kTmemCols);
    const int64_t m = mlp_batch_size(p);
    // shrinking threshold T: the caller's value or the batch mean; every CTA adds the losses in the same order
    double T_shrink = (double)p.threshold;
    if (p.thresh_mode != AA_THRESH_VALUE) {
        double acc = 0.0;
        for (int64_t i = tid; i < m; i += kStepMlpThreads) acc += (double)__ldg(p.loss + i);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) red[warp] = acc;
    }
    volatile int* abort_flag = &tp->abort_flag;
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (p.thresh_mode != AA_THRESH_VALUE) {
        double total = 0.0;
        for (int wi = 0; wi < kStepMlpThreads / 32; ++wi) total += red[wi];
        T_shrink = m > 0 ? total / (double)m : 0.0;
    }
    const uint32_t tmem_base = *(volatile uint32_t*)&tp->tmem_base;
    const unsigned int n_tiles = (unsigned int)((m + kHalfRows - 1) / kHalfRows);

    if (warp == 0) {
        if (!mlp_produce<GATHER, kHalfRows, kHalfStages>(tp, ring, &map_x, &map_w, p.g, n_tiles, p.row_idx, m, p.n_stored) && lane == 0) step_give_up(p, tp);
    } else if (GATHER && (warp == 3 || warp >= 12)) {
        if (!mlp_produce<GATHER, kHalfRows, kHalfStages>(tp, ring, &map_x, &map_w, p.g, n_tiles, p.row_idx, m, p.n_stored, warp == 3 ? 1 : warp - 10) && lane == 0)
            step_give_up(p, tp);
    } else if (warp == 1) {
        if (!mlp_issue_mma<kHalfRows, kHalfStages>(tp, ring, p.g, n_tiles, tmem_base) && lane == 0) step_give_up(p, tp);
    } else if (warp >= 4 && warp < 12) {
        // ------------------------------------------------------------ epilogue
        // warps 4..7 take this CTA's even tiles (accumulator 0), warps 8..11 the odd ones (accumulator 1)
        const int ew = warp - 4;
        const int quad = warp & 3, acc = ew >> 2;
        const int row = quad * 32 + lane;
        const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * kMaxHidden);
        const float bias2 = *p.b2;
        float sum_rh[kMaxHidden / 32], sum_p[kMaxHidden / 32];   // lane l: columns c0 + l of this warp's rows
#pragma unroll
        for (int c = 0; c < kMaxHidden / 32; ++c) sum_rh[c] = sum_p[c] = 0.0f;
        float sum_r = 0.0f;
        int it = acc;
        for (unsigned long long tile = blockIdx.x + (unsigned long long)acc * gridDim.x; tile < n_tiles; tile += 2ull * gridDim.x, it += 2) {
            if (!mbar_wait(&tp->acc_full[acc], (uint32_t)((it >> 1) & 1), abort_flag)) {
                if (lane == 0) step_give_up(p, tp);
                break;
            }
            tc_fence_after_sync();
            const int64_t i = (int64_t)tile * kHalfRows + row;
            // this row's loss and validity are requested before the pass over TMEM
            bool valid = i < m;
            float f_i = 0.0f;
            if (valid) {
                f_i = __ldg(p.loss + i);
                if (GATHER && (unsigned long long)(long long)p.row_idx[i] >= (unsigned long long)p.n_stored) {
                    latch(p.ctl, AA_ERR_BAD_INDEX);
                    valid = false;
                }
            }
            float s = 0.0f;
            for (int c0 = 0; c0 < hidden; c0 += 32) {
                uint32_t a[32];
                tmem_ld_32cols(t_row + (uint32_t)c0, a);
                tmem_ld_wait();
                // hidden is a multiple of 16: the accumulator columns past it were never written and may hold anything
                if (c0 + 32 > hidden) {
#pragma unroll
                    for (int q = 16; q < 32; ++q) a[q] = 0u;
                }
#pragma unroll
                for (int q = 0; q < 32; ++q) s = fmaf(fmaxf(__uint_as_float(a[q]) + b1_s[c0 + q], 0.0f), w2_s[c0 + q], s);
            }
            float r = 0.0f;
            if (valid) {
                const float z = (double)f_i > T_shrink ? 1.0f : 0.0f;
                r = sigmoid_f32(s + bias2) - z;
            }
            sum_r += r;
            {
                // r as two bf16 terms: the W1-gradient contraction multiplies each of them with the rows
                const __nv_bfloat16 hi = __float2bfloat16_rn(r);
                p.r_hi[i] = hi;
                p.r_lo[i] = __float2bfloat16_rn(r - __bfloat162float(hi));
            }
            // gate words of this warp's 32 rows (adjacent in i): word (i >> 5) & 1 of block i >> 6
            uint32_t* gate_dst = p.gate_bits + (((int64_t)tile * kHalfRows + quad * 32) >> 6) * (2 * kMaxHidden) + (quad & 1);
#pragma unroll
            for (int c = 0; c < kMaxHidden / 32; ++c) {
                const int c0 = c * 32;
                if (c0 < hidden) {
                    uint32_t a[32];
                    tmem_ld_32cols(t_row + (uint32_t)c0, a);
                    tmem_ld_wait();
                    if (c0 + 32 > hidden) {
#pragma unroll
                        for (int q = 16; q < 32; ++q) a[q] = 0u;
                    }
                    float rh[32], pm[32];
                    uint32_t mine = 0;
#pragma unroll
                    for (int q = 0; q < 32; ++q) {
                        const float pre = __uint_as_float(a[q]) + b1_s[c0 + q];
                        const bool on = pre > 0.0f;
                        rh[q] = on ? r * pre : 0.0f;
                        pm[q] = on ? r : 0.0f;
                        const uint32_t gates = __ballot_sync(0xFFFFFFFFu, on);   // unit c0 + q over the warp's rows
                        if (lane == q) mine = gates;
                    }
                    gate_dst[(c0 + lane) * 2] = mine;
                    sum_rh[c] += lanes_transpose_sum(rh, lane);
                    sum_p[c] += lanes_transpose_sum(pm, lane);
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tp->acc_empty[acc]);
        }
#pragma unroll
        for (int c = 0; c < kMaxHidden / 32; ++c) {
            col_s[(ew * 2 + 0) * kMaxHidden + c * 32 + lane] = sum_rh[c];
            col_s[(ew * 2 + 1) * kMaxHidden + c * 32 + lane] = sum_p[c];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum_r += __shfl_xor_sync(0xFFFFFFFFu, sum_r, o);
        if (lane == 0) rsum_s[ew] = sum_r;
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 2) tmem_dealloc(tmem_base, kTmemCols);
    // this CTA's column sums, warps added in a fixed order
    float* out = p.small + (int64_t)blockIdx.x * (2 * kMaxHidden + 1);
    for (int j = tid; j < 2 * kMaxHidden; j += kStepMlpThreads) {
        const int which = j / kMaxHidden, u = j % kMaxHidden;
        float t = 0.0f;
        for (int w = 0; w < kStepEpiWarps; ++w) t += col_s[(w * 2 + which) * kMaxHidden + u];
        out[j] = t;
    }
    if (tid == 0) {
        float t = 0.0f;
        for (int w = 0; w < kStepEpiWarps; ++w) t += rsum_s[w];
        out[2 * kMaxHidden] = t;
    }
}

// ---------------------------------------------------------------- residuals from the screening's scores and gates
constexpr int kPrepThreads = 512;
constexpr int kPrepWarps = kPrepThreads / 32;

// Transpose of a 32 x 32 bit matrix held one row per lane (bit c of lane i's word = element [i][c]): five rounds of
// block swaps between lanes j apart.  Afterwards bit i of lane c's word is element [i][c].
__device__ __forceinline__ uint32_t warp_bit_transpose(uint32_t x, int lane) {
    const uint32_t masks[5] = {0x0000FFFFu, 0x00FF00FFu, 0x0F0F0F0Fu, 0x33333333u, 0x55555555u};
#pragma unroll
    for (int step = 0; step < 5; ++step) {
        const int j = 16 >> step;
        const uint32_t m = masks[step];
        const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, x, j);
        // lanes with bit j clear keep their low blocks and take the partner's low blocks into their high ones;
        // the partner does the opposite
        x = (lane & j) ? ((x & ~m) | ((other >> j) & m)) : ((x & m) | ((other & m) << j));
    }
    return x;
}

__global__ void __launch_bounds__(kPrepThreads, 1) mlp_prepare_kernel(MlpStepParams p) {
    __shared__ double red[kPrepWarps];
    __shared__ float col_s[kPrepWarps][kMaxHidden];      // per warp: sum_i r_i [a_iu > 0]
    __shared__ float tab_s[kPrepWarps][8][16];           // per warp: sums of r over every subset of each 4-row group
    __shared__ float rsum_s[kPrepWarps];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t m = mlp_batch_size(p);
    // shrinking threshold T: the caller's value or the batch mean; every CTA adds the losses in the same order
    double T_shrink = (double)p.threshold;
    if (p.thresh_mode != AA_THRESH_VALUE) {
        double acc = 0.0;
        if (((uintptr_t)p.loss & 15) == 0) {
            const int64_t quads = m >> 2;
            for (int64_t q = tid; q < quads; q += kPrepThreads) {
                const float4 v = __ldg(reinterpret_cast<const float4*>(p.loss) + q);
                acc += ((double)v.x + (double)v.y) + ((double)v.z + (double)v.w);
            }
            for (int64_t i = (quads << 2) + tid; i < m; i += kPrepThreads) acc += (double)__ldg(p.loss + i);
        } else {
            for (int64_t i = tid; i < m; i += kPrepThreads) acc += (double)__ldg(p.loss + i);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) red[warp] = acc;
        __syncthreads();
        double total = 0.0;
        for (int wi = 0; wi < kPrepWarps; ++wi) total += red[wi];
        T_shrink = m > 0 ? total / (double)m : 0.0;
    }
    float sum_p[kMaxHidden / 32];                        // lane l: units c * 32 + l over this warp's rows
#pragma unroll
    for (int c = 0; c < kMaxHidden / 32; ++c) sum_p[c] = 0.0f;
    float sum_r = 0.0f;
    // groups of 32 adjacent batch rows, up to the end of the last 64-row slice the W1-gradient kernel reads
    const int64_t n_groups = ((m + kRowSlice - 1) / kRowSlice) * (kRowSlice / 32);
    for (int64_t g = (int64_t)blockIdx.x * kPrepWarps + warp; g < n_groups; g += (int64_t)gridDim.x * kPrepWarps) {
        const int64_t i = g * 32 + lane;
        bool valid = i < m;
        long long row = 0;
        if (valid) {
            row = p.row_idx ? (long long)p.row_idx[i] : (long long)i;
            if ((unsigned long long)row >= (unsigned long long)p.n_stored) {
                latch(p.ctl, AA_ERR_BAD_INDEX);
                valid = false;
            }
        }
        float r = 0.0f;
        uint4 g_lo = make_uint4(0, 0, 0, 0), g_hi = make_uint4(0, 0, 0, 0);
        if (valid) {
            const float f_i = __ldg(p.loss + i);
            const float z = (double)f_i > T_shrink ? 1.0f : 0.0f;
            r = sigmoid_f32(__ldg(p.score + row)) - z;
            const uint4* src = reinterpret_cast<const uint4*>(p.gate_cand + row * (kMaxHidden / 32));
            g_lo = __ldg(src);
            g_hi = __ldg(src + 1);
        }
        sum_r += r;
        {
            const __nv_bfloat16 hi = __float2bfloat16_rn(r);
            p.r_hi[i] = hi;
            p.r_lo[i] = __float2bfloat16_rn(r - __bfloat162float(hi));
        }
        // Table for the column sums: entry [k][s] = sum of r over the rows 4 k + b of this group whose bit b is set in s.
        // Lane l fills the four entries [l >> 2][4 (l & 3) .. + 3].
        {
            const int k = lane >> 2;
            const float r0 = __shfl_sync(0xFFFFFFFFu, r, 4 * k), r1 = __shfl_sync(0xFFFFFFFFu, r, 4 * k + 1);
            const float r2 = __shfl_sync(0xFFFFFFFFu, r, 4 * k + 2), r3 = __shfl_sync(0xFFFFFFFFu, r, 4 * k + 3);
            const float high = ((lane & 1) ? r2 : 0.0f) + ((lane & 2) ? r3 : 0.0f);      // bits 2 and 3 of s = lane & 3
            __syncwarp();                                   // the previous group's look-ups are done
            float* t = &tab_s[warp][k][4 * (lane & 3)];
            t[0] = high;
            t[1] = r0 + high;
            t[2] = r1 + high;
            t[3] = (r0 + r1) + high;
            __syncwarp();
        }
        const uint32_t words[kMaxHidden / 32] = {g_lo.x, g_lo.y, g_lo.z, g_lo.w, g_hi.x, g_hi.y, g_hi.z, g_hi.w};
        uint32_t* gate_dst = p.gate_bits + (g >> 1) * (2 * kMaxHidden) + (g & 1);
#pragma unroll
        for (int c = 0; c < kMaxHidden / 32; ++c) {
            if (c * 32 < p.g.hidden) {
                // lane q ends with unit c * 32 + q over the warp's rows
                const uint32_t mine = warp_bit_transpose(words[c], lane);
                gate_dst[(c * 32 + lane) * 2] = mine;
                float acc = 0.0f;
#pragma unroll
                for (int k = 0; k < 8; ++k) acc += tab_s[warp][k][(mine >> (4 * k)) & 15u];
                sum_p[c] += acc;
            }
        }
    }
#pragma unroll
    for (int c = 0; c < kMaxHidden / 32; ++c) col_s[warp][c * 32 + lane] = sum_p[c];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum_r += __shfl_xor_sync(0xFFFFFFFFu, sum_r, o);
    if (lane == 0) rsum_s[warp] = sum_r;
    __syncthreads();
    float* out = p.small + (int64_t)blockIdx.x * (2 * kMaxHidden + 1);
    if (tid < kMaxHidden) {
        float t = 0.0f;
        for (int w = 0; w < kPrepWarps; ++w) t += col_s[w][tid];
        out[tid] = 0.0f;                                  // grad w2 comes from the W1-gradient partials on this route
        out[kMaxHidden + tid] = t;
    }
    if (tid == 0) {
        float t = 0.0f;
        for (int w = 0; w < kPrepWarps; ++w) t += rsum_s[w];
        out[2 * kMaxHidden] = t;
    }
}

// ---------------------------------------------------------------- G = P^T X over the batch rows
constexpr int kXStages = 3;                                     // ring of feature-row slices (TMA)
constexpr uint32_t kATileBytes = kMaxHidden * 128;              // one term of P^T for a slice: up to 256 units x 64 rows, bf16
constexpr uint32_t kXChunkBytes = kRowSlice * 128;              // 64 batch rows x 64 feature columns
constexpr uint32_t kXStageBytes = 4 * kXChunkBytes;             // 256 feature columns
constexpr int kBuildWarps = 8;                                  // warps 4..11 build the P^T tiles, then drain the accumulators

constexpr int kATiles = 4;                                      // ring of P^T tiles: r_hi and r_lo tiles of two slices
struct GradPipe {
    uint64_t x_full[kXStages], x_empty[kXStages];
    uint64_t a_full[kATiles], a_empty[kATiles];
    uint64_t acc_full, drain;
    uint32_t tmem_base;
    int abort_flag;
    uint32_t gate_lut[16];     // four gate bits (4 batch rows of one unit) -> two byte-permute selectors, see below
};

// prmt selector that keeps (bit set) or zeroes (bit clear) each 16-bit half of a word holding two bf16 values:
// bit 0 -> low half, bit 1 -> high half; a zeroed byte is taken from the permute's second operand (0).
__device__ __forceinline__ uint32_t pair_selector(uint32_t two_bits) {
    return ((two_bits & 1u) ? 0x0010u : 0x0044u) | ((two_bits & 2u) ? 0x3200u : 0x4400u);
}
__device__ __forceinline__ uint32_t gate_pair(uint32_t pair, uint32_t selector) {
    uint32_t out;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(out) : "r"(pair), "r"(0u), "r"(selector));
    return out;
}

template <bool GATHER>
__global__ void __launch_bounds__(kStepMlpThreads, 1)
mlp_w1_grad_kernel(const __grid_constant__ CUtensorMap map_x, MlpStepParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring_x = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char* ring_a = ring_x + (size_t)kXStages * kXStageBytes;           // [kATiles][kATileBytes]: tile 2 sl + term, modulo the ring
    GradPipe* gp = reinterpret_cast<GradPipe*>(ring_a + (size_t)kATiles * kATileBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kXStages; ++s) {
            mbar_init(&gp->x_full[s], 1);
            mbar_init(&gp->x_empty[s], 1);
        }
        for (int b = 0; b < kATiles; ++b) {
            mbar_init(&gp->a_full[b], kBuildWarps);
            mbar_init(&gp->a_empty[b], 1);
        }
        mbar_init(&gp->acc_full, 1);
        mbar_init(&gp->drain, 1);
        gp->abort_flag = 0;
        mbar_fence_init();
        prefetch_tensormap(&map_x);
    }
    if (warp == 2) tmem_alloc(&gp->tmem_base, kTmemCols);
    if (tid < 16) {
        // entry b: the selectors of row pairs (0,1) and (2,3), 16 bits each
        const uint32_t b = (uint32_t)tid;
        gp->gate_lut[tid] = pair_selector(b & 3u) | (pair_selector((b >> 2) & 3u) << 16);
    }
    volatile int* abort_flag = &gp->abort_flag;
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *(volatile uint32_t*)&gp->tmem_base;

    const int64_t m = mlp_batch_size(p);
    const int chunk = blockIdx.x % p.n_chunks, split = blockIdx.x / p.n_chunks;
    const int64_t total_slices = (m + kRowSlice - 1) / kRowSlice;
    const int64_t per = (total_slices + p.splits - 1) / p.splits;
    const int64_t s_begin = (int64_t)split * per;
    const int64_t s_end = s_begin + per < total_slices ? s_begin + per : total_slices;
    const int n_slices = s_end > s_begin ? (int)(s_end - s_begin) : 0;
    const int col0 = chunk * kFeatChunk;
    int n_q = (int)((p.d - col0 + 63) / 64);           // 64-column feature chunks that exist
    if (n_q > 4) n_q = 4;
    const int hidden = p.g.hidden;
    const bool two_halves = hidden > 128;

    if (warp == 0 || (GATHER && (warp == 3 || warp >= 12))) {
        // ------------------------------------------------------------ producer (warp 0) and, for gathered rows, seven helpers:
        // gather warp q fetches rows (q & 1) * 32 .. + 32 of 64-column chunk q >> 1 of every stage, eight four-row gathers
        // (one per issuing lane); warp 0 also posts the expected bytes.
        const int part = warp == 0 ? 0 : (warp == 3 ? 1 : warp - 10);
        const int chunk_q = part >> 1, half = part & 1;
        int stage = 0, j = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int sl = 0; sl < n_slices; ++sl) {
            const int64_t i0 = (s_begin + sl) * kRowSlice;
            int r0 = 0, r1 = 0, r2 = 0, r3 = 0;
            if (GATHER && lane < 8) {
                int rr[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int64_t i = i0 + half * 32 + lane * 4 + q;
                    long long row = i < m ? (long long)p.row_idx[i] : 0;
                    if ((unsigned long long)row >= (unsigned long long)p.n_stored) row = 0;   // its r is zero
                    rr[q] = (int)row;
                }
                r0 = rr[0]; r1 = rr[1]; r2 = rr[2]; r3 = rr[3];
            }
            if (!mbar_wait(&gp->x_empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
            unsigned char* x_dst = ring_x + (size_t)stage * kXStageBytes;
            if (lane == 0 && part == 0) {
                mbar_arrive_expect_tx(&gp->x_full[stage], (uint32_t)n_q * kXChunkBytes);
                if (!GATHER)
                    for (int q = 0; q < n_q; ++q) tma_load_2d(x_dst + q * kXChunkBytes, &map_x, col0 + q * 64, (int)i0, &gp->x_full[stage]);
            }
            if (GATHER) {
                __syncwarp();
                if (lane < 8 && chunk_q < n_q)
                    tma_gather4(x_dst + chunk_q * kXChunkBytes + (half * 32 + lane * 4) * 128, &map_x, col0 + chunk_q * 64, r0, r1, r2, r3,
                                &gp->x_full[stage]);
            }
            __syncwarp();
            ++j;
            if (++stage == kXStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) {
            if (lane == 0) { latch(p.ctl, AA_ERR_SCAN_TIMEOUT); *abort_flag = 1; }
            const int pending = j < kXStages ? j : kXStages;
            for (int back = 1; back <= pending; ++back) {
                const int jj = j - back, st = jj % kXStages, use = jj / kXStages;
                const long long t0 = clock64();
                while (!mbar_try_wait(&gp->x_full[st], (uint32_t)(use & 1)) && clock64() - t0 < kWaitCycles) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        const uint32_t idesc = umma_idesc_bf16(128, kFeatChunk, false, true);   // A = P^T K-major, B = feature rows MN-major
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int sl = 0; sl < n_slices && ok; ++sl) {
            if (!mbar_wait(&gp->x_full[stage], phase, abort_flag)) { ok = false; break; }
            const uint32_t b_addr = smem_u32(ring_x + (size_t)stage * kXStageBytes);
#pragma unroll
            for (int term = 0; term < 2; ++term) {                      // r_hi, then r_lo, into the same accumulators
                const int tile = 2 * sl + term, q = tile & (kATiles - 1);
                if (!mbar_wait(&gp->a_full[q], (uint32_t)((tile / kATiles) & 1), abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                if (lane == 0) {
                    const uint32_t a_addr = smem_u32(ring_a + (size_t)q * kATileBytes);
#pragma unroll
                    for (int k = 0; k < kRowSlice / 16; ++k) {
                        // 16 batch rows = two 8-row groups (1024 bytes apart); 64-column chunks are 8192 bytes apart
                        const uint64_t b_desc = umma_smem_desc(b_addr + k * 2048, kXChunkBytes, 1024);
                        const bool acc = (sl | k | term) != 0;
                        umma_bf16(tmem_base, umma_smem_desc(a_addr + k * 32, 16, 1024), b_desc, idesc, acc);
                        if (two_halves) umma_bf16(tmem_base + kFeatChunk, umma_smem_desc(a_addr + 128 * 128 + k * 32, 16, 1024), b_desc, idesc, acc);
                    }
                    umma_commit(&gp->a_empty[q]);
                    if (term == 1) {
                        umma_commit(&gp->x_empty[stage]);
                        if (sl == n_slices - 1) umma_commit(&gp->acc_full);
                    }
                }
                __syncwarp();
            }
            if (++stage == kXStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok && lane == 0) { latch(p.ctl, AA_ERR_SCAN_TIMEOUT); *abort_flag = 1; }
        if (lane == 0) umma_commit(&gp->drain);
        __syncwarp();
        const long long t0 = clock64();
        while (!mbar_try_wait(&gp->drain, 0) && clock64() - t0 < kWaitCycles) {}
    } else if (warp >= 4 && warp < 12) {
        // ------------------------------------------------------------ builders: P^T tiles of every slice from the gate bits and r
        // Thread (cq, ub): the 16-byte chunk cq (batch rows 8 cq .. 8 cq + 7 of the slice) of units ub, ub + 32, ...
        // Tile layout = what a 128-byte-swizzled TMA box [units x 64 rows] would be: unit u at u * 128 bytes, its chunk cq at
        // position cq ^ (u & 7) within the 128-byte row.
        const int bt = tid - 128;
        const int cq = bt & 7, ub = bt >> 3;
        constexpr int kUnitTrips = kMaxHidden / 32;
        const uint32_t row_off = (uint32_t)((ub >> 3) * 1024 + (ub & 7) * 128 + ((cq ^ (ub & 7)) << 4));
        uint32_t gates[kUnitTrips];
        uint4 rh = make_uint4(0, 0, 0, 0), rl = make_uint4(0, 0, 0, 0);
        auto fetch = [&](int sl) {
            const int64_t block = s_begin + sl;
            const uint32_t* src = p.gate_bits + block * (2 * kMaxHidden) + (cq >> 2);
#pragma unroll
            for (int t = 0; t < kUnitTrips; ++t) gates[t] = (ub + 32 * t) < hidden ? __ldg(src + (ub + 32 * t) * 2) : 0u;
            rh = __ldg(reinterpret_cast<const uint4*>(p.r_hi + block * kRowSlice) + cq);
            rl = __ldg(reinterpret_cast<const uint4*>(p.r_lo + block * kRowSlice) + cq);
        };
        bool ok = true;
        if (n_slices > 0) fetch(0);
        for (int sl = 0; sl < n_slices && ok; ++sl) {
            // selectors of this thread's chunk for every unit it serves: one table look-up per gate byte
            uint2 sel[kUnitTrips];
#pragma unroll
            for (int t = 0; t < kUnitTrips; ++t) {
                const uint32_t gb = gates[t] >> ((cq & 3) * 8);
                sel[t] = make_uint2(gp->gate_lut[gb & 0xFu], gp->gate_lut[(gb >> 4) & 0xFu]);
            }
            const uint4 r_term[2] = {rh, rl};
            if (sl + 1 < n_slices) fetch(sl + 1);            // next slice's words are in flight while this one is built
#pragma unroll
            for (int term = 0; term < 2; ++term) {
                const int tile = 2 * sl + term, q = tile & (kATiles - 1);
                if (!mbar_wait(&gp->a_empty[q], (uint32_t)(((tile / kATiles) & 1) ^ 1), abort_flag)) { ok = false; break; }
                unsigned char* a_tile = ring_a + (size_t)q * kATileBytes + row_off;
                const uint4 rv = r_term[term];
#pragma unroll
                for (int t = 0; t < kUnitTrips; ++t) {
                    if (ub + 32 * t < hidden)
                        *reinterpret_cast<uint4*>(a_tile + t * 4096) =
                            make_uint4(gate_pair(rv.x, sel[t].x), gate_pair(rv.y, sel[t].x >> 16), gate_pair(rv.z, sel[t].y), gate_pair(rv.w, sel[t].y >> 16));
                }
                // the tensor cores read shared memory through the asynchronous proxy: order these plain stores before it
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(&gp->a_full[q]);
            }
        }
        if (!ok && lane == 0) { latch(p.ctl, AA_ERR_SCAN_TIMEOUT); *abort_flag = 1; }
        // ------------------------------------------------------------ epilogue: this CTA's partial of G
        const int quad = warp & 3, acc = (warp - 4) >> 2;
        const int u = acc * 128 + quad * 32 + lane;                 // hidden unit
        const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * kFeatChunk);
        bool have = ok && n_slices > 0 && (acc == 0 || two_halves);
        if (ok && n_slices > 0 && !mbar_wait(&gp->acc_full, 0, abort_flag)) {
            if (lane == 0) { latch(p.ctl, AA_ERR_SCAN_TIMEOUT); *abort_flag = 1; }
            have = false;
        }
        tc_fence_after_sync();
        float* dst = p.part + ((int64_t)split * p.g.hidden + u) * p.d_pad + col0;
        for (int c0 = 0; c0 < kFeatChunk; c0 += 32) {
            uint32_t v[32];
            if (have) {
                tmem_ld_32cols(t_row + (uint32_t)c0, v);
                tmem_ld_wait();
            } else {
#pragma unroll
                for (int q = 0; q < 32; ++q) v[q] = 0u;
            }
            if (u < p.g.hidden && col0 + c0 < p.d_pad) {
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    reinterpret_cast<float4*>(dst + c0)[q] = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                                                        __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 2) tmem_dealloc(tmem_base, kTmemCols);
}

// ---------------------------------------------------------------- updates
__global__ void __launch_bounds__(256) mlp_apply_w1_kernel(MlpStepParams p) {
    const int64_t m = mlp_batch_size(p);
    if (m <= 0) return;
    const float scale = p.lr / (float)m;
    const float inv_m = 1.0f / (float)m;
    if ((p.d & 3) == 0 && (p.d_pad & 3) == 0 && (((uintptr_t)p.W1 | (uintptr_t)p.part) & 15) == 0 && ((uintptr_t)p.W1_bf16 & 7) == 0) {
        // four adjacent feature columns per thread: 16-byte loads of the split-K partials and of W1
        const int64_t dq = p.d >> 2, total = (int64_t)p.g.hidden * dq;
        for (int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; q < total; q += (int64_t)gridDim.x * blockDim.x) {
            const int64_t u = q / dq, k = (q - u * dq) << 2;
            float4 g = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll 4
            for (int s = 0; s < p.splits; ++s) {
                const float4 t = __ldcs(reinterpret_cast<const float4*>(p.part + ((int64_t)s * p.g.hidden + u) * p.d_pad + k));
                g.x += t.x; g.y += t.y; g.z += t.z; g.w += t.w;
            }
            const float w2u = __ldg(p.w2 + u);
            float4* wp = reinterpret_cast<float4*>(p.W1 + u * p.d + k);
            float4 w = *wp;
            const float gv[4] = {g.x, g.y, g.z, g.w};
            if (p.gw2_part) {
                // sum_k W1b_uk G_uk over this warp's 128 columns of unit u (d is a multiple of 128 on this route, so the
                // 32 lanes share u), with the bf16 weights the screening multiplied with
                const uint2 wb = *reinterpret_cast<const uint2*>(p.W1_bf16 + u * p.d + k);
                float dot = __uint_as_float(wb.x << 16) * g.x;
                dot = fmaf(__uint_as_float(wb.x & 0xFFFF0000u), g.y, dot);
                dot = fmaf(__uint_as_float(wb.y << 16), g.z, dot);
                dot = fmaf(__uint_as_float(wb.y & 0xFFFF0000u), g.w, dot);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xFFFFFFFFu, dot, o);
                if ((threadIdx.x & 31) == 0) p.gw2_part[u * p.gw2_segs + (k >> 7)] = dot;
            }
            float wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int e = 0; e < 4; ++e)
                wv[e] = p.adam.on ? adam_update(p.adam, wv[e], w2u * gv[e] * inv_m, p.lr, u * p.d + k + e) : wv[e] - scale * w2u * gv[e];
            *wp = make_float4(wv[0], wv[1], wv[2], wv[3]);
            __nv_bfloat162 lo = __floats2bfloat162_rn(wv[0], wv[1]), hi = __floats2bfloat162_rn(wv[2], wv[3]);
            uint2 packed;
            packed.x = *reinterpret_cast<uint32_t*>(&lo);
            packed.y = *reinterpret_cast<uint32_t*>(&hi);
            *reinterpret_cast<uint2*>(p.W1_bf16 + u * p.d + k) = packed;
        }
        return;
    }
    const int64_t total = (int64_t)p.g.hidden * p.d;
    for (int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; q < total; q += (int64_t)gridDim.x * blockDim.x) {
        const int64_t u = q / p.d, k = q - u * p.d;
        float g = 0.0f;
        for (int s = 0; s < p.splits; ++s) g += p.part[((int64_t)s * p.g.hidden + u) * p.d_pad + k];
        const float w = p.adam.on ? adam_update(p.adam, p.W1[q], __ldg(p.w2 + u) * g * inv_m, p.lr, q)
                                  : p.W1[q] - scale * __ldg(p.w2 + u) * g;
        p.W1[q] = w;
        p.W1_bf16[q] = __float2bfloat16_rn(w);
    }
}

// b1, w2, b2 from the per-CTA column sums: kSmallSlices thread rows share the CTAs (loads in flight together), the
// slices are added in a fixed order.
constexpr int kSmallSlices = 4;
__global__ void __launch_bounds__(kMaxHidden * kSmallSlices) mlp_apply_small_kernel(MlpStepParams p, int ctas) {
    __shared__ float part_w2[kSmallSlices][kMaxHidden], part_b1[kSmallSlices][kMaxHidden], part_b2[32];
    const int64_t m = mlp_batch_size(p);
    if (m <= 0) return;
    const float scale = p.lr / (float)m;
    const int u = threadIdx.x % kMaxHidden, slice = threadIdx.x / kMaxHidden;
    {
        float g_w2 = 0.0f, g_b1 = 0.0f;
#pragma unroll 8
        for (int c = slice; c < ctas; c += kSmallSlices) {
            const float* in = p.small + (int64_t)c * (2 * kMaxHidden + 1);
            g_w2 += in[u];
            g_b1 += in[kMaxHidden + u];
        }
        part_w2[slice][u] = g_w2;
        part_b1[slice][u] = g_b1;
    }
    if (threadIdx.x < 32) {
        float g_b2 = 0.0f;
        for (int c = threadIdx.x; c < ctas; c += 32) g_b2 += p.small[(int64_t)c * (2 * kMaxHidden + 1) + 2 * kMaxHidden];
        part_b2[threadIdx.x] = g_b2;
    }
    __syncthreads();
    if (slice == 0 && u < p.g.hidden) {
        float g_w2 = 0.0f, g_b1 = 0.0f;
#pragma unroll
        for (int q = 0; q < kSmallSlices; ++q) {
            g_w2 += part_w2[q][u];
            g_b1 += part_b1[q][u];
        }
        if (p.gw2_part) {
            // sum_i r_i relu(a_iu) = sum_k W1b_uk G_uk + b1_u sum_i r_i [a_iu > 0]  (b1 still holds the old value)
            float t = 0.0f;
            for (int seg = 0; seg < p.gw2_segs; ++seg) t += p.gw2_part[u * p.gw2_segs + seg];
            g_w2 = fmaf(p.b1[u], g_b1, t);
        }
        const float w2_old = p.w2[u];
        const int64_t hd = (int64_t)p.g.hidden * p.d;      // moments: W1, then b1, w2, b2
        if (p.adam.on) {
            p.b1[u] = adam_update(p.adam, p.b1[u], w2_old * g_b1 / (float)m, p.lr, hd + u);
            p.w2[u] = adam_update(p.adam, w2_old, g_w2 / (float)m, p.lr, hd + p.g.hidden + u);
        } else {
            p.b1[u] = p.b1[u] - scale * w2_old * g_b1;
            p.w2[u] = w2_old - scale * g_w2;
        }
    }
    if (threadIdx.x == 0) {
        float g_b2 = 0.0f;
        for (int q = 0; q < 32; ++q) g_b2 += part_b2[q];
        p.b2[0] = p.adam.on ? adam_update(p.adam, p.b2[0], g_b2 / (float)m, p.lr, (int64_t)p.g.hidden * p.d + 2 * p.g.hidden)
                            : p.b2[0] - scale * g_b2;
    }
}

}  // namespace

constexpr size_t kSmallBytes = ((size_t)kMaxMlpCtas * (2 * kMaxHidden + 1) * 4 + 255) / 256 * 256;

size_t mlp_step_workspace_bytes(int64_t max_rows, int64_t max_d, int64_t max_hidden, size_t* pt_bytes, size_t* small_bytes,
                                size_t* gate_off) {
    const size_t pitch = (size_t)((max_rows + kSuperRows - 1) / kSuperRows * kSuperRows);
    // what the residual kernel hands to the W1-gradient kernel: gate bits (256 units per row = 32 bytes) and r as two bf16
    // terms; behind it the gate words the last screening left for every row of its pool (32 bytes per row)
    *gate_off = (pitch * (kMaxHidden / 8 + 4) + 255) / 256 * 256;
    *pt_bytes = *gate_off + (pitch * (kMaxHidden / 8) + 255) / 256 * 256;
    // per-CTA column sums, then the per-warp dot products of the grad-w2 identity ([kMaxHidden][max_d / 128])
    *small_bytes = kSmallBytes + ((size_t)kMaxHidden * (size_t)((max_d + 127) / 128) * 4 + 255) / 256 * 256;
    // split-K partials: chunks * splits <= kMaxMlpCtas CTAs, each [hidden x 256] fp32 (+ one chunk of slack per split row)
    const size_t d_pad = (size_t)((max_d + kFeatChunk - 1) / kFeatChunk * kFeatChunk);
    const size_t n_chunks = d_pad / kFeatChunk;
    size_t splits = kMaxMlpCtas / n_chunks;
    if (splits < 1) splits = 1;
    return splits * (size_t)max_hidden * d_pad * 4;
}

aa_status launch_assistant_step_mlp(aa_ctx_impl* c, const MlpFeat& f, float* W1_master, const int32_t* row_idx, int64_t n_stored,
                                    int64_t m_host, const int32_t* count_dev, const float* loss, float lr, int thresh_mode,
                                    float threshold) {
    if (m_host <= 0) return AA_OK;
    if (f.hidden < 16 || f.hidden > kMaxHidden || f.hidden % 16) return AA_ERR_UNSUPPORTED;
    if ((uintptr_t)f.x % 16 || (f.row_stride * 2) % 16 || (uintptr_t)f.W1_bf16 % 16 || (f.d * 2) % 16) return AA_ERR_UNSUPPORTED;
    if (!c->mlp_pt || m_host > c->max_rows || f.d > c->max_d || f.hidden > c->max_hidden) return AA_ERR_WORKSPACE;
    const bool gather = row_idx != nullptr;
    MlpStepParams p = {};
    p.row_idx = row_idx;
    p.n_stored = n_stored;
    p.m_host = m_host;
    p.count_dev = count_dev;
    p.loss = loss;
    p.thresh_mode = thresh_mode;
    p.threshold = threshold;
    p.lr = lr;
    p.W1 = W1_master;
    p.W1_bf16 = static_cast<__nv_bfloat16*>(const_cast<void*>(f.W1_bf16));
    p.b1 = const_cast<float*>(f.b1);
    p.w2 = const_cast<float*>(f.w2);
    p.b2 = const_cast<float*>(f.b2);
    p.d = f.d;
    p.g = make_mlp_geom(f.d, f.hidden, kHalfRows);
    p.pitch = (m_host + kSuperRows - 1) / kSuperRows * kSuperRows;
    p.gate_bits = static_cast<uint32_t*>(c->mlp_pt);
    p.r_hi = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(c->mlp_pt) + (size_t)p.pitch * (kMaxHidden / 8));
    p.r_lo = p.r_hi + p.pitch;
    p.small = c->mlp_small;
    p.part = c->mlp_part;
    p.d_pad = (f.d + kFeatChunk - 1) / kFeatChunk * kFeatChunk;
    p.n_chunks = (int)(p.d_pad / kFeatChunk);
    p.adam = c->adam;
    p.ctl = c->ctl;
    int max_ctas = c->sm_count < kMaxMlpCtas ? c->sm_count : kMaxMlpCtas;
    if (p.n_chunks > max_ctas) return AA_ERR_UNSUPPORTED;
    const int64_t slices = (m_host + kRowSlice - 1) / kRowSlice;
    int64_t splits = max_ctas / p.n_chunks;
    if (splits > slices) splits = slices;
    if (splits < 1) splits = 1;
    while (splits > 1 && (size_t)splits * (size_t)f.hidden * (size_t)p.d_pad * 4 > c->mlp_part_bytes) --splits;
    if ((size_t)splits * (size_t)f.hidden * (size_t)p.d_pad * 4 > c->mlp_part_bytes) return AA_ERR_WORKSPACE;
    p.splits = (int)splits;
    // The screening's scores and gates stand in for the forward pass when they are the ones of these rows under these
    // weights: the caller passed scores, the last two-layer screening on this context ran on this very pool (no candidate
    // list) with this W1, and no update has gone through the context since.
    const bool scored = c->step_score && c->mlp_gate_cand && c->gate_feat == f.x && c->gate_w1 == f.W1_bf16 && c->gate_n == f.n &&
                        n_stored == f.n && f.d % 128 == 0 && (uintptr_t)W1_master % 16 == 0;
    c->gate_feat = nullptr;      // the parameters change below: the gates in the workspace go stale
    if (scored) {
        p.score = c->step_score;
        p.gate_cand = c->mlp_gate_cand;
        p.gw2_part = reinterpret_cast<float*>(reinterpret_cast<char*>(c->mlp_small) + kSmallBytes);
        p.gw2_segs = (int)(f.d / 128);
    }

    alignas(64) CUtensorMap map_x, map_w, map_xg;
    if (!encode_bf16_tile_map(&map_x, f.x, (uint64_t)f.n, (uint64_t)f.d, (uint64_t)f.row_stride, gather ? 1 : kHalfRows) ||
        !encode_bf16_tile_map(&map_w, f.W1_bf16, (uint64_t)f.hidden, (uint64_t)f.d, (uint64_t)f.d, (uint32_t)f.hidden) ||
        !encode_bf16_tile_map(&map_xg, f.x, (uint64_t)f.n, (uint64_t)f.d, (uint64_t)f.row_stride, gather ? 1 : kRowSlice))
        return AA_ERR_CUDA;

    // 1. forward + residuals + P^T
    {
        const size_t smem = 1024 + (size_t)kHalfStages * p.g.stage_bytes + sizeof(float) * (2 * kMaxHidden + kStepEpiWarps * 2 * kMaxHidden) +
                            sizeof(double) * (kStepMlpThreads / 32) + sizeof(float) * kStepEpiWarps + sizeof(TilePipe) + 64;
        const void* kernel = gather ? (const void*)mlp_residual_kernel<true> : (const void*)mlp_residual_kernel<false>;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return AA_ERR_CUDA;
        const int64_t tiles = (m_host + kHalfRows - 1) / kHalfRows;
        int grid = max_ctas;
        if (grid > tiles) grid = (int)tiles;
        if (scored) {
            const int64_t groups = (m_host + kRowSlice - 1) / kRowSlice * (kRowSlice / 32);
            grid = max_ctas;
            if (grid > (groups + kPrepWarps - 1) / kPrepWarps) grid = (int)((groups + kPrepWarps - 1) / kPrepWarps);
            void* args[] = {&p};
            if (cudaLaunchKernel((const void*)mlp_prepare_kernel, dim3(grid), dim3(kPrepThreads), args, 0, c->stream) != cudaSuccess)
                return AA_ERR_CUDA;
        } else {
            void* args[] = {&map_x, &map_w, &p};
            if (cudaLaunchKernel(kernel, dim3(grid), dim3(kStepMlpThreads), args, smem, c->stream) != cudaSuccess) return AA_ERR_CUDA;
        }
        ++c->launches;
        // 2. G = P^T X
        const size_t smem2 = 1024 + (size_t)kXStages * kXStageBytes + (size_t)kATiles * kATileBytes + sizeof(GradPipe) + 64;
        const void* k2 = gather ? (const void*)mlp_w1_grad_kernel<true> : (const void*)mlp_w1_grad_kernel<false>;
        if (cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2) != cudaSuccess) return AA_ERR_CUDA;
        void* args2[] = {&map_xg, &p};
        if (cudaLaunchKernel(k2, dim3(p.n_chunks * p.splits), dim3(kStepMlpThreads), args2, smem2, c->stream) != cudaSuccess)
            return AA_ERR_CUDA;
        ++c->launches;
        // 3. updates (W1 first: it reads the old w2)
        void* args3[] = {&p};
        const int64_t total = f.hidden * f.d;
        int agrid = (int)((total / 4 + 255) / 256);
        if (agrid > c->sm_count * 8) agrid = c->sm_count * 8;
        if (agrid < 1) agrid = 1;
        if (cudaLaunchKernel((const void*)mlp_apply_w1_kernel, dim3(agrid), dim3(256), args3, 0, c->stream) != cudaSuccess) return AA_ERR_CUDA;
        ++c->launches;
        void* args4[] = {&p, &grid};
        if (cudaLaunchKernel((const void*)mlp_apply_small_kernel, dim3(1), dim3(kMaxHidden * kSmallSlices), args4, 0, c->stream) != cudaSuccess)
            return AA_ERR_CUDA;
        ++c->launches;
    }
    return AA_OK;
}

}  // namespace aa
