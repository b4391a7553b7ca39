// Assistant labels + one SGD step (Sec. "Learning to generate smart training batches" label rule and objective; Algorithm 2:
// Assistant.gradient, Assistant.update) for the linear Assistant g = sigmoid(w.x + b).
//
// Dense features: each CTA stages a block of batch rows in shared memory once, computes
// their residuals r_i = g_i - z_i (one warp per row) and then adds r_i x_i into column
// accumulators that stay in registers for the whole kernel (each thread owns fixed
// columns).  CTAs write their column sums to a partial buffer; a second small kernel adds
// the partials in a fixed order and applies  w <- w - lr * grad,  so the result does not
// depend on scheduling.  CSR features: residuals first, then a scatter of -lr/M r_i val
// onto the touched weights with fp32 atomics.
#include <math.h>

#include "step_common.cuh"

namespace aa {

namespace {

// ---------------------------------------------------------------- dense
// CI = 16-byte column vectors owned by each thread.  VEC = rows are 16-byte aligned.
template <typename T, int CI, bool VEC>
__global__ void __launch_bounds__(kStepThreads) linear_grad_dense_kernel(StepParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int VE = Vec<T>::kElems;
    __shared__ double red[kStepWarps];
    __shared__ float res[32];              // residual per staged row
    float* w_s = reinterpret_cast<float*>(smem_raw);                 // [d_pad]
    T* x_s = reinterpret_cast<T*>(smem_raw + p.d_pad * sizeof(float));   // [rows_per_block][d_pad]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t d = p.f.d, d_pad = p.d_pad;
    const int nvec = (int)(d_pad / VE);
    const int RB = p.rows_per_block;
    const int64_t m = batch_size(p);
    const double T_shrink = block_threshold(p, m, red);

    for (int64_t j = tid; j < d_pad; j += kStepThreads) w_s[j] = j < d ? p.f.w[j] : 0.0f;
    const float bias = *p.f.b;
    const T* base = static_cast<const T*>(p.f.base);

    float acc[CI][VE];
#pragma unroll
    for (int ci = 0; ci < CI; ++ci)
#pragma unroll
        for (int e = 0; e < VE; ++e) acc[ci][e] = 0.0f;
    float bias_acc = 0.0f;   // used by lane 0 of each warp

    const int64_t n_blocks = (m + RB - 1) / RB;
    for (int64_t blk = blockIdx.x; blk < n_blocks; blk += gridDim.x) {
        const int64_t i0 = blk * RB;
        __syncthreads();   // previous block's readers are done (and w_s is complete)
        // stage the rows
        if (VEC) {
            for (int q = tid; q < RB * nvec; q += kStepThreads) {
                const int rl = q / nvec, v = q - rl * nvec;
                const int64_t i = i0 + rl;
                uint4 val = make_uint4(0, 0, 0, 0);
                if (i < m) {
                    const long long r = batch_row(p, i);
                    if (r >= 0) val = __ldg(reinterpret_cast<const uint4*>(base + r * p.f.row_stride) + v);
                }
                reinterpret_cast<uint4*>(x_s + (int64_t)rl * d_pad)[v] = val;
            }
        } else {
            for (int64_t q = tid; q < (int64_t)RB * d_pad; q += kStepThreads) {
                const int rl = (int)(q / d_pad);
                const int64_t j = q - (int64_t)rl * d_pad;
                const int64_t i = i0 + rl;
                T val = T(0);
                if (i < m && j < d) {
                    const long long r = batch_row(p, i);
                    if (r >= 0) val = base[r * p.f.row_stride + j];
                }
                x_s[(int64_t)rl * d_pad + j] = val;
            }
        }
        __syncthreads();
        // residuals, one warp per staged row
        for (int rl = warp; rl < RB; rl += kStepWarps) {
            const int64_t i = i0 + rl;
            float dot = 0.0f;
            const T* xr = x_s + (int64_t)rl * d_pad;
            for (int v = lane; v < nvec; v += 32) {
                float x[VE];
                Vec<T>::unpack(reinterpret_cast<const uint4*>(xr)[v], x);
                const float* wp = w_s + (int64_t)v * VE;
#pragma unroll
                for (int e = 0; e < VE; ++e) dot = fmaf(x[e], wp[e], dot);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xFFFFFFFFu, dot, o);
            if (lane == 0) {
                float r = 0.0f;
                if (i < m) {
                    const float z = (double)__ldg(p.loss + i) > T_shrink ? 1.0f : 0.0f;
                    r = sigmoid_f32(dot + bias) - z;
                    if (p.row_idx && (unsigned long long)(long long)p.row_idx[i] >= (unsigned long long)p.n_stored) r = 0.0f;
                    bias_acc += r;
                }
                res[rl] = r;
            }
        }
        __syncthreads();
        // column sums: acc += r_i * x_i
#pragma unroll
        for (int ci = 0; ci < CI; ++ci) {
            const int v = tid + ci * kStepThreads;
            if (v < nvec) {
                for (int rl = 0; rl < RB; ++rl) {
                    const float r = res[rl];
                    float x[VE];
                    Vec<T>::unpack(reinterpret_cast<const uint4*>(x_s + (int64_t)rl * d_pad)[v], x);
#pragma unroll
                    for (int e = 0; e < VE; ++e) acc[ci][e] = fmaf(r, x[e], acc[ci][e]);
                }
            }
        }
    }

    // this CTA's column sums and bias sum
    float* part = p.partials + (int64_t)blockIdx.x * d_pad;
#pragma unroll
    for (int ci = 0; ci < CI; ++ci) {
        const int v = tid + ci * kStepThreads;
        if (v < nvec) {
#pragma unroll
            for (int e = 0; e < VE; ++e) part[(int64_t)v * VE + e] = acc[ci][e];
        }
    }
    __syncthreads();
    float* bred = reinterpret_cast<float*>(red);
    if (lane == 0) bred[warp] = bias_acc;
    __syncthreads();
    if (tid == 0) {
        float t = 0.0f;
        for (int wi = 0; wi < kStepWarps; ++wi) t += bred[wi];
        p.partials[(int64_t)gridDim.x * d_pad + blockIdx.x] = t;
    }
}

// Adds the partials and applies the SGD update.  A CTA owns 32 columns; its 8 warps each add a
// strided share of the partials (loads in flight, not a serial chain) and the 8 shares are then
// combined in a fixed order, so the result is reproducible for a given set of partials.
__global__ void __launch_bounds__(256) linear_apply_kernel(StepParams p, int parts) {
    __shared__ float share[8][33];
    const int64_t m = batch_size(p);
    if (m <= 0) return;
    const float scale = p.lr / (float)m;
    const int lane = threadIdx.x & 31, grp = threadIdx.x >> 5;
    const int64_t j = (int64_t)blockIdx.x * 32 + lane;
    float g = 0.0f;
    if (j < p.f.d) {
#pragma unroll 4
        for (int q = grp; q < parts; q += 8) g += p.partials[(int64_t)q * p.d_pad + j];
    }
    share[grp][lane] = g;
    __syncthreads();
    if (grp == 0 && j < p.f.d) {
        float t = 0.0f;
#pragma unroll
        for (int k = 0; k < 8; ++k) t += share[k][lane];
        p.w[j] = p.adam.on ? adam_update(p.adam, p.w[j], t / (float)m, p.lr, j) : p.w[j] - scale * t;
    }
    if (blockIdx.x == 0 && grp == 1) {
        // bias: the per-CTA residual sums sit behind the column partials
        float t = 0.0f;
        for (int q = lane; q < parts; q += 32) t += p.partials[(int64_t)parts * p.d_pad + q];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
        if (lane == 0) p.b[0] = p.adam.on ? adam_update(p.adam, p.b[0], t / (float)m, p.lr, p.f.d) : p.b[0] - scale * t;
    }
}

// ---------------------------------------------------------------- CSR
constexpr int kCsrStepUnroll = 8;
template <int LPR>
__global__ void __launch_bounds__(256) csr_residual_kernel(StepParams p) {
    __shared__ double red[8];
    const int64_t m = batch_size(p);
    const double T_shrink = block_threshold(p, m, red);
    const float bias = *p.csr.b;
    const int gl = threadIdx.x % LPR;
    const int64_t groups = (int64_t)gridDim.x * (blockDim.x / LPR);
    const int64_t g0 = (int64_t)blockIdx.x * (blockDim.x / LPR) + threadIdx.x / LPR;
    const int64_t rounds = (m + groups - 1) / groups;
    for (int64_t it = 0; it < rounds; ++it) {
        const int64_t i = g0 + it * groups;
        const long long r = i < m ? batch_row(p, i) : -1;
        float acc = 0.0f;
        if (r >= 0) {
            const int e0 = __ldg(p.csr.indptr + r), e1 = __ldg(p.csr.indptr + r + 1);
            // kCsrStepUnroll entries per lane and trip: their loads, then their weight gathers, are in flight together
            for (int e = e0 + gl; e < e1; e += kCsrStepUnroll * LPR) {
                int c[kCsrStepUnroll];
                float v[kCsrStepUnroll], wq[kCsrStepUnroll];
#pragma unroll
                for (int u = 0; u < kCsrStepUnroll; ++u) {
                    const int ee = e + u * LPR;
                    const bool in = ee < e1;
                    c[u] = in ? __ldg(p.csr.col + ee) : 0;
                    v[u] = in ? __ldg(p.csr.val + ee) : 0.0f;
                }
                bool bad = false;
#pragma unroll
                for (int u = 0; u < kCsrStepUnroll; ++u) {
                    const bool ok = (unsigned long long)(unsigned int)c[u] < (unsigned long long)p.csr.d;
                    bad |= !ok;
                    wq[u] = ok ? p.w[c[u]] : 0.0f;
                }
#pragma unroll
                for (int u = 0; u < kCsrStepUnroll; ++u) acc = fmaf(v[u], wq[u], acc);
                if (bad) latch(p.ctl, AA_ERR_BAD_INDEX);
            }
        }
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (gl == 0 && i < m) {
            float res = 0.0f;
            if (r >= 0) {
                const float z = (double)__ldg(p.loss + i) > T_shrink ? 1.0f : 0.0f;
                res = sigmoid_f32(acc + bias) - z;
            }
            p.residual[i] = res;
        }
    }
}

template <int LPR>
__global__ void __launch_bounds__(256) csr_scatter_kernel(StepParams p) {
    const int64_t m = batch_size(p);
    if (m <= 0) return;
    // SGD adds -lr/M r_i val straight onto the weights; Adam needs the mean gradient itself, collected in the
    // (cleared) partial buffer and applied by adam_dense_kernel.
    const float scale = p.adam.on ? 1.0f / (float)m : -p.lr / (float)m;
    float* w_dst = p.adam.on ? p.partials : p.w;
    float* b_dst = p.adam.on ? p.partials + p.csr.d : p.b;
    const int gl = threadIdx.x % LPR;
    const int64_t groups = (int64_t)gridDim.x * (blockDim.x / LPR);
    const int64_t g0 = (int64_t)blockIdx.x * (blockDim.x / LPR) + threadIdx.x / LPR;
    const int64_t rounds = (m + groups - 1) / groups;
    float bias_acc = 0.0f;
    for (int64_t it = 0; it < rounds; ++it) {
        const int64_t i = g0 + it * groups;
        if (i >= m) continue;
        const long long r = p.row_idx ? (long long)p.row_idx[i] : i;
        if ((unsigned long long)r >= (unsigned long long)p.n_stored) continue;   // latched by the residual pass
        const float step = scale * p.residual[i];
        if (gl == 0) bias_acc += step;
        const int e0 = __ldg(p.csr.indptr + r), e1 = __ldg(p.csr.indptr + r + 1);
        for (int e = e0 + gl; e < e1; e += kCsrStepUnroll * LPR) {
            int c[kCsrStepUnroll];
            float v[kCsrStepUnroll];
#pragma unroll
            for (int u = 0; u < kCsrStepUnroll; ++u) {
                const int ee = e + u * LPR;
                const bool in = ee < e1;
                c[u] = in ? __ldg(p.csr.col + ee) : -1;
                v[u] = in ? __ldg(p.csr.val + ee) : 0.0f;
            }
#pragma unroll
            for (int u = 0; u < kCsrStepUnroll; ++u)
                if ((unsigned long long)(unsigned int)c[u] < (unsigned long long)p.csr.d) atomicAdd(w_dst + c[u], step * v[u]);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) bias_acc += __shfl_xor_sync(0xFFFFFFFFu, bias_acc, o);
    if ((threadIdx.x & 31) == 0 && bias_acc != 0.0f) atomicAdd(b_dst, bias_acc);
}

// Adam over every weight of the bag-of-words Assistant from the mean gradient in the partial buffer (a weight whose
// gradient is zero still moves while its first moment decays).
__global__ void __launch_bounds__(256) adam_dense_kernel(StepParams p) {
    const int64_t m = batch_size(p);
    if (m <= 0) return;
    const int64_t d = p.csr.d;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j <= d; j += (int64_t)gridDim.x * blockDim.x) {
        float* param = j < d ? p.w + j : p.b;
        *param = adam_update(p.adam, *param, p.partials[j], p.lr, j);
    }
}

template <typename T, bool VEC>
const void* pick_dense_kernel(int ci) {
    switch (ci) {
        case 1: return (const void*)linear_grad_dense_kernel<T, 1, VEC>;
        case 2: return (const void*)linear_grad_dense_kernel<T, 2, VEC>;
        case 4: return (const void*)linear_grad_dense_kernel<T, 4, VEC>;
        default: return (const void*)linear_grad_dense_kernel<T, 8, VEC>;
    }
}

}  // namespace

aa_status launch_linear_apply(aa_ctx_impl* c, const StepParams& p_in, int parts) {
    StepParams p = p_in;
    void* args[] = {&p, &parts};
    const int agrid = (int)((p.f.d + 31) / 32);
    if (cudaLaunchKernel((const void*)linear_apply_kernel, dim3(agrid), dim3(256), args, 0, c->stream) != cudaSuccess)
        return AA_ERR_CUDA;
    ++c->launches;
    return AA_OK;
}

aa_status launch_assistant_step_dense(aa_ctx_impl* c, const DenseFeat& f, const int32_t* row_idx, int64_t n_stored,
                                      int64_t m_host, const int32_t* count_dev, const float* loss, float* w, float* b,
                                      float lr, int thresh_mode, float threshold) {
    if (m_host <= 0) return AA_OK;
    const int es = f.dtype == AA_BF16 ? 2 : 4;
    const int ve = 16 / es;
    const bool vec = ((uintptr_t)f.base % 16 == 0) && ((f.row_stride * es) % 16 == 0) && (f.d % ve == 0);
    StepParams p = {};
    p.f = f;
    p.row_idx = row_idx;
    p.n_stored = n_stored;
    p.m_host = m_host;
    p.count_dev = count_dev;
    p.loss = loss;
    p.score = c->step_score;      // used by the matrix-instruction kernel; the other kernels recompute the pre-activations
    p.thresh_mode = thresh_mode;
    p.threshold = threshold;
    p.lr = lr;
    p.w = w;
    p.b = b;
    p.partials = c->partials;
    p.adam = c->adam;
    p.ctl = c->ctl;
    p.d_pad = (f.d + ve - 1) / ve * ve;
    if (vec) {
        int parts = 0;
        aa_status st = p.score ? launch_assistant_grad_dense_scored(c, p, &parts) : AA_ERR_UNSUPPORTED;
        if (st == AA_OK) return AA_OK;
        if (st != AA_ERR_UNSUPPORTED) return st;
        st = launch_assistant_grad_dense_mma(c, p, &parts);
        if (st == AA_OK) return parts > 0 ? launch_linear_apply(c, p, parts) : AA_OK;
        if (st != AA_ERR_UNSUPPORTED) return st;
        st = launch_assistant_grad_dense_tma(c, p, &parts);
        if (st == AA_OK) return launch_linear_apply(c, p, parts);
        if (st != AA_ERR_UNSUPPORTED) return st;
    }
    const int64_t nvec = p.d_pad / ve;
    int ci = 1;
    while (ci < 8 && (int64_t)ci * kStepThreads < nvec) ci <<= 1;
    if ((int64_t)ci * kStepThreads < nvec) return AA_ERR_UNSUPPORTED;   // dense rows beyond 4096 vectors

    // rows staged per block: as many as fit in ~64 KB beside w, between 1 and 32
    const int64_t row_bytes = p.d_pad * es;
    int64_t rb = (64 * 1024) / row_bytes;
    rb = rb < 1 ? 1 : (rb > 32 ? 32 : rb);
    p.rows_per_block = (int)rb;
    const size_t smem = (size_t)p.d_pad * sizeof(float) + (size_t)rb * row_bytes;
    if (smem > 200 * 1024) return AA_ERR_UNSUPPORTED;

    const void* kernel = f.dtype == AA_BF16 ? (vec ? pick_dense_kernel<uint16_t, true>(ci) : pick_dense_kernel<uint16_t, false>(ci))
                                            : (vec ? pick_dense_kernel<float, true>(ci) : pick_dense_kernel<float, false>(ci));
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return AA_ERR_CUDA;
    int grid = resident_ctas(c, kernel, kStepThreads, smem);
    if (grid <= 0) return AA_ERR_CUDA;
    const int64_t n_blocks = (m_host + rb - 1) / rb;
    if (grid > n_blocks) grid = (int)n_blocks;
    const int64_t max_parts = c->partial_floats / (p.d_pad + 1);
    if (max_parts < 1) return AA_ERR_WORKSPACE;
    if (grid > max_parts) grid = (int)max_parts;
    if (grid > kMaxParts) grid = kMaxParts;

    void* args[] = {&p};
    if (cudaLaunchKernel(kernel, dim3(grid), dim3(kStepThreads), args, smem, c->stream) != cudaSuccess) return AA_ERR_CUDA;
    ++c->launches;
    return launch_linear_apply(c, p, grid);
}

aa_status launch_assistant_step_csr(aa_ctx_impl* c, const CsrFeat& f, const int32_t* row_idx, int64_t n_stored,
                                    int64_t m_host, const int32_t* count_dev, const float* loss, float* w, float* b,
                                    float lr, int thresh_mode, float threshold) {
    if (m_host <= 0) return AA_OK;
    if (m_host > c->max_rows) return AA_ERR_WORKSPACE;
    StepParams p = {};
    p.csr = f;
    p.row_idx = row_idx;
    p.n_stored = n_stored;
    p.m_host = m_host;
    p.count_dev = count_dev;
    p.loss = loss;
    p.thresh_mode = thresh_mode;
    p.threshold = threshold;
    p.lr = lr;
    p.w = w;
    p.b = b;
    p.residual = c->row_scratch;
    p.partials = c->partials;
    p.adam = c->adam;
    p.ctl = c->ctl;
    if (p.adam.on) {
        if (f.d + 1 > c->partial_floats) return AA_ERR_WORKSPACE;
        if (cudaMemsetAsync(c->partials, 0, sizeof(float) * (size_t)(f.d + 1), c->stream) != cudaSuccess) return AA_ERR_CUDA;
    }
    int lpr = 4;   // about one unrolled trip per lane for a row of average length
    while (lpr < 32 && (float)lpr * kCsrStepUnroll * 1.1f < f.mean_nnz) lpr <<= 1;
    const int64_t rows_per_cta = 256 / lpr;
    const int64_t want = (m_host + rows_per_cta - 1) / rows_per_cta;
    const int cap = c->sm_count * 8;
    const int grid = (int)(want < cap ? want : cap);
    void* args[] = {&p};
    const void* k1;
    const void* k2;
    switch (lpr) {
        case 4: k1 = (const void*)csr_residual_kernel<4>; k2 = (const void*)csr_scatter_kernel<4>; break;
        case 8: k1 = (const void*)csr_residual_kernel<8>; k2 = (const void*)csr_scatter_kernel<8>; break;
        case 16: k1 = (const void*)csr_residual_kernel<16>; k2 = (const void*)csr_scatter_kernel<16>; break;
        default: k1 = (const void*)csr_residual_kernel<32>; k2 = (const void*)csr_scatter_kernel<32>; break;
    }
    if (cudaLaunchKernel(k1, dim3(grid), dim3(256), args, 0, c->stream) != cudaSuccess) return AA_ERR_CUDA;
    ++c->launches;
    if (cudaLaunchKernel(k2, dim3(grid), dim3(256), args, 0, c->stream) != cudaSuccess) return AA_ERR_CUDA;
    ++c->launches;
    if (p.adam.on) {
        const int64_t want = (f.d + 1 + 255) / 256;
        const int agrid = (int)(want < c->sm_count * 8 ? want : c->sm_count * 8);
        if (cudaLaunchKernel((const void*)adam_dense_kernel, dim3(agrid), dim3(256), args, 0, c->stream) != cudaSuccess) return AA_ERR_CUDA;
        ++c->launches;
    }
    return AA_OK;
}

}  // namespace aa
