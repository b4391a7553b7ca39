// Assistant gradient for 16-byte aligned dense rows (Sec. "Learning to generate smart training batches" objective; Algorithm 2:
// Assistant.gradient), as one persistent, warp-specialised CTA per SM fed by bulk copies.
//
//   producer warp : takes tickets of batch rows and streams them (gathered through the batch
//                   list, one cp.async.bulk per row, or one per stage when rows are adjacent)
//                   into a shared-memory ring.
//   dot warps     : per stage, the pre-activation of each row under the current parameters,
//                   the label z = 1[loss > T] and the residual r = sigmoid(s) - z.
//   column warps  : every thread owns fixed feature columns for the whole kernel and adds
//                   r_i * x_i for each staged row into registers; they release the stage.
//
// Each row is read from HBM once.  CTAs write their column sums to the partial buffer; the
// apply kernel adds the partials and takes the SGD step.  Rows are handed out dynamically, so
// the summation order (not the result beyond rounding) can differ between runs.
#include "async_copy.cuh"
#include "step_common.cuh"

namespace aa {

namespace {

constexpr int kGMaxStages = 8;
constexpr int kDotWarps = 8;
constexpr int kDotSplit = 2;                          // dot warps sharing one stage
constexpr int kDotPairs = kDotWarps / kDotSplit;      // stage j goes to pair j % kDotPairs
constexpr int kColWarps = 12;
constexpr int kColThreads = kColWarps * 32;
constexpr int kWorkWarps = kDotWarps + kColWarps;
constexpr int kGradThreads = (1 + kWorkWarps) * 32;   // warp 0 producer, 1..8 dot, 9..20 column
constexpr int kGMaxRowBytes = 24 * 1024;
constexpr int kGTargetStage = 24 * 1024;
constexpr int kTicketRows = 32;                       // batch rows per ticket: one row index per producer lane

struct GradGeometry {
    int chunk_rows;       // rows per stage (power of two <= 32)
    int stage_bytes;
    int stages;
    int split;            // dot warps per stage in use (1 or 2)
    int contiguous;
    int nvec;
    uint32_t row_bytes;
};

struct GradControl {
    uint64_t x_full[kGMaxStages], r_full[kGMaxStages], x_empty[kGMaxStages];
    long long first_row[kGMaxStages];     // batch position of the stage's first row
    float r[kGMaxStages][32];             // residual per staged row (0 = skip the row)
    unsigned int valid[kGMaxStages];      // bit i: row i of the stage was fetched
    double red[kWorkWarps];
    float bias_sum;
    int stop_j;
    int abort_flag;
};

__device__ __forceinline__ void grad_give_up(const StepParams& p, GradControl* cb) {
    latch(p.ctl, AA_ERR_SCAN_TIMEOUT);
    *(volatile int*)&cb->abort_flag = 1;
}

// Pre-activation lane-partials of one or two staged rows (all 32 lanes on each row).
template <typename T>
__device__ __forceinline__ void dot_pair(const uint4* r0, const uint4* r1, const float* w_s, int nvec, int lane, float& a0, float& a1) {
    constexpr int VE = Vec<T>::kElems;
    float p0[VE], p1[VE];
#pragma unroll
    for (int e = 0; e < VE; ++e) p0[e] = p1[e] = 0.0f;
#pragma unroll 4
    for (int v = lane; v < nvec; v += 32) {
        float x0[VE], x1[VE], wq[VE];
        Vec<T>::unpack(r0[v], x0);
        Vec<T>::unpack(r1[v], x1);
        Vec<T>::load_w(w_s, nvec, v, wq);
#pragma unroll
        for (int e = 0; e < VE; ++e) {
            p0[e] = fmaf(x0[e], wq[e], p0[e]);
            p1[e] = fmaf(x1[e], wq[e], p1[e]);
        }
    }
    a0 = a1 = 0.0f;
#pragma unroll
    for (int e = 0; e < VE; ++e) {
        a0 += p0[e];
        a1 += p1[e];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a0 += __shfl_xor_sync(0xFFFFFFFFu, a0, o);
        a1 += __shfl_xor_sync(0xFFFFFFFFu, a1, o);
    }
}

template <typename T, int CI>
__global__ void __launch_bounds__(kGradThreads, 1) linear_grad_tma_kernel(StepParams p, GradGeometry g) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int VE = Vec<T>::kElems;
    unsigned char* x_ring = smem;
    float* w_s = reinterpret_cast<float*>(smem + (size_t)g.stages * g.stage_bytes);
    GradControl* cb = reinterpret_cast<GradControl*>(w_s + (size_t)g.nvec * VE);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < g.stages; ++s) {
            mbar_init(&cb->x_full[s], 1);
            mbar_init(&cb->r_full[s], (uint32_t)g.split);
            mbar_init(&cb->x_empty[s], kColWarps);
        }
        cb->bias_sum = 0.0f;
        cb->stop_j = 0x7FFFFFFF;
        cb->abort_flag = 0;
        mbar_fence_init();
    }
    const int64_t m = batch_size(p);
    volatile int* abort_flag = &cb->abort_flag;
    __syncthreads();   // barriers are initialised

    // While the producer already streams rows, all other warps stage the weights and add up the
    // batch losses for the mean threshold (fixed order: per-thread stride, warp tree, warp index).
    if (warp >= 1) {
        const int wt = tid - 32;
#pragma unroll 4
        for (int jj = wt; jj < p.f.d; jj += kWorkWarps * 32) w_s[Vec<T>::w_index(jj, g.nvec)] = p.f.w[jj];
        if (p.thresh_mode != AA_THRESH_VALUE) {
            double acc = 0.0;
            int64_t head = 0;
            if (((uintptr_t)p.loss & 15) == 0) {
                const int64_t nv = m / 4;
                const float4* lv = reinterpret_cast<const float4*>(p.loss);
#pragma unroll 4
                for (int64_t v = wt; v < nv; v += kWorkWarps * 32) {
                    const float4 q = __ldg(lv + v);
                    acc += ((double)q.x + (double)q.y) + ((double)q.z + (double)q.w);
                }
                head = nv * 4;
            }
            for (int64_t i = head + wt; i < m; i += kWorkWarps * 32) acc += (double)__ldg(p.loss + i);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
            if (lane == 0) cb->red[warp - 1] = acc;
        }
        asm volatile("bar.sync 2, %0;" ::"n"(kWorkWarps * 32) : "memory");
    }

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        const unsigned char* base = static_cast<const unsigned char*>(p.f.base);
        const size_t stride_bytes = (size_t)p.f.row_stride * sizeof(T);
        const int spt = kTicketRows / g.chunk_rows;   // stages per ticket
        const unsigned int n_tickets = (unsigned int)((m + kTicketRows - 1) / kTicketRows);
        int j = 0, stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        // Software pipeline over tickets: while ticket `cur` is issued, the row indices of `next`
        // and the ticket after it are already on their way, so no stage waits on a global load.
        auto fetch_row = [&](unsigned int tk) -> long long {
            const int64_t i = (int64_t)tk * kTicketRows + lane;
            if (tk >= n_tickets || i >= m) return -1;
            return g.contiguous ? (long long)i : batch_row(p, i);
        };
        unsigned int cur = 0, next = 0;
        if (lane == 0) cur = atomicAdd(&p.ctl->ticket, 1u);
        cur = __shfl_sync(0xFFFFFFFFu, cur, 0);
        long long cur_row = fetch_row(cur);
        if (lane == 0) next = atomicAdd(&p.ctl->ticket, 1u);
        while (ok && cur < n_tickets) {
            next = __shfl_sync(0xFFFFFFFFu, next, 0);
            const long long next_row = fetch_row(next);
            unsigned int after = 0;
            if (lane == 0) after = atomicAdd(&p.ctl->ticket, 1u);
            for (int s = 0; s < spt; ++s) {
                const int64_t i0 = (int64_t)cur * kTicketRows + (int64_t)s * g.chunk_rows;
                if (i0 >= m) break;
                if (j >= g.stages && !mbar_wait(&cb->x_empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                unsigned char* dst = x_ring + (size_t)stage * g.stage_bytes;
                const long long r = __shfl_sync(0xFFFFFFFFu, cur_row, (s * g.chunk_rows + lane) & 31);
                const bool mine = lane < g.chunk_rows && r >= 0;
                const unsigned int have = __ballot_sync(0xFFFFFFFFu, mine);
                if (lane == 0) {
                    cb->first_row[stage] = i0;
                    cb->valid[stage] = have;
                }
                if (g.contiguous) {
                    if (lane == 0) {
                        const uint32_t bytes = (uint32_t)__popc(have) * g.row_bytes;   // valid rows are a prefix
                        mbar_arrive_expect_tx(&cb->x_full[stage], bytes);
                        bulk_g2s(dst, base + (size_t)i0 * stride_bytes, bytes, &cb->x_full[stage]);
                    }
                } else {
                    if (lane == 0) {
                        if (have) mbar_arrive_expect_tx(&cb->x_full[stage], (uint32_t)__popc(have) * g.row_bytes);
                        else mbar_arrive(&cb->x_full[stage]);
                    }
                    __syncwarp();
                    if (mine) bulk_g2s(dst + (size_t)lane * g.row_bytes, base + (size_t)r * stride_bytes, g.row_bytes, &cb->x_full[stage]);
                }
                __syncwarp();
                ++j;
                if (++stage == g.stages) { stage = 0; phase ^= 1u; }
            }
            cur = next;
            cur_row = next_row;
            next = after;
        }
        if (ok) {
            // One empty stage per dot pair wakes every pair; the pair that owns the first of them
            // passes the stop on to the column warps.  Each of these stages was last used by a
            // real chunk, which the column warps release before they see the stop.
            if (lane == 0) *(volatile int*)&cb->stop_j = j;
            for (int c = 0; c < kDotPairs && ok; ++c) {
                if (j >= g.stages && !mbar_wait(&cb->x_empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                if (lane == 0) mbar_arrive(&cb->x_full[stage]);
                ++j;
                if (++stage == g.stages) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok) {
            if (lane == 0) grad_give_up(p, cb);
            const int pending = j < g.stages ? j : g.stages;
            for (int back = 1; back <= pending; ++back) {
                const int jj = j - back, st = jj % g.stages, use = jj / g.stages;
                const long long t0 = clock64();
                while (!mbar_try_wait(&cb->x_full[st], (uint32_t)(use & 1)) && clock64() - t0 < kWaitCycles) {}
            }
        }
    } else if (warp <= kDotWarps) {
        // ------------------------------------------------------------ dot warps
        const int dw = warp - 1;
        // shrinking threshold T: the caller's value, or the batch mean from the staged partial sums
        double T_shrink = (double)p.threshold;
        if (p.thresh_mode != AA_THRESH_VALUE) {
            double total = 0.0;
            for (int wi = 0; wi < kWorkWarps; ++wi) total += cb->red[wi];
            T_shrink = m > 0 ? total / (double)m : 0.0;
        }
        const float bias = *p.f.b;
        const int pair = dw / kDotSplit, part = dw % kDotSplit;
        float bias_acc = 0.0f;
        if (part < g.split) {
            const int rows_per = g.chunk_rows / g.split;
            for (int j = pair;; j += kDotPairs) {
                const int stage = j % g.stages, use = j / g.stages;
                if (!mbar_wait(&cb->x_full[stage], (uint32_t)(use & 1), abort_flag)) {
                    if (lane == 0) grad_give_up(p, cb);
                    break;
                }
                if (j >= *(volatile int*)&cb->stop_j) {
                    if (lane == 0) mbar_arrive(&cb->r_full[stage]);   // hands the stop to the column warps
                    break;
                }
                const int64_t i0 = cb->first_row[stage];
                const unsigned int valid_rows = cb->valid[stage];
                const unsigned char* xs = x_ring + (size_t)stage * g.stage_bytes;
                for (int rl = part * rows_per; rl < (part + 1) * rows_per; rl += 2) {
                    const int rl1 = rl + 1 < (part + 1) * rows_per ? rl + 1 : rl;
                    // lanes 0 and 1 own the two rows; their loss is requested before the dot product
                    const int row = lane == 0 ? rl : rl1;
                    const bool valid = lane < 2 && (lane == 0 || rl1 != rl) && ((valid_rows >> row) & 1u);
                    float f_i = 0.0f;
                    if (valid) f_i = __ldg(p.loss + i0 + row);
                    float a0, a1;
                    dot_pair<T>(reinterpret_cast<const uint4*>(xs + (size_t)rl * g.row_bytes),
                                reinterpret_cast<const uint4*>(xs + (size_t)rl1 * g.row_bytes), w_s, g.nvec, lane, a0, a1);
                    if (lane < 2 && (lane == 0 || rl1 != rl)) {
                        float res = 0.0f;
                        if (valid) {
                            const float z = (double)f_i > T_shrink ? 1.0f : 0.0f;
                            res = sigmoid_f32((lane == 0 ? a0 : a1) + bias) - z;
                            bias_acc += res;
                        }
                        cb->r[stage][row] = res;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&cb->r_full[stage]);
            }
        }
        bias_acc += __shfl_xor_sync(0xFFFFFFFFu, bias_acc, 1);
        if (lane == 0 && bias_acc != 0.0f) atomicAdd(&cb->bias_sum, bias_acc);
    } else {
        // ------------------------------------------------------------ column warps
        const int ct = tid - (1 + kDotWarps) * 32;
        float acc[CI][VE];
#pragma unroll
        for (int ci = 0; ci < CI; ++ci)
#pragma unroll
            for (int e = 0; e < VE; ++e) acc[ci][e] = 0.0f;
        for (int j = 0;; ++j) {
            const int stage = j % g.stages, use = j / g.stages;
            if (!mbar_wait(&cb->r_full[stage], (uint32_t)(use & 1), abort_flag)) {
                if (lane == 0) grad_give_up(p, cb);
                break;
            }
            if (j >= *(volatile int*)&cb->stop_j) break;
            const unsigned char* xs = x_ring + (size_t)stage * g.stage_bytes;
            for (int rl = 0; rl < g.chunk_rows; ++rl) {
                const float r = cb->r[stage][rl];
                if (r != 0.0f) {   // 0 marks rows past the batch end or unreadable rows (their stage bytes are stale)
#pragma unroll
                    for (int ci = 0; ci < CI; ++ci) {
                        const int v = ct + ci * kColThreads;
                        if (v < g.nvec) {
                            float x[VE];
                            Vec<T>::unpack(reinterpret_cast<const uint4*>(xs + (size_t)rl * g.row_bytes)[v], x);
#pragma unroll
                            for (int e = 0; e < VE; ++e) acc[ci][e] = fmaf(r, x[e], acc[ci][e]);
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&cb->x_empty[stage]);
        }
        float* part = p.partials + (int64_t)blockIdx.x * p.d_pad;
#pragma unroll
        for (int ci = 0; ci < CI; ++ci) {
            const int v = ct + ci * kColThreads;
            if (v < g.nvec) {
#pragma unroll
                for (int e = 0; e < VE; ++e) part[(int64_t)v * VE + e] = acc[ci][e];
            }
        }
    }
    __syncthreads();
    if (tid == 0) {
        p.partials[(int64_t)gridDim.x * p.d_pad + blockIdx.x] = cb->bias_sum;
        // last CTA out re-arms the ticket counter for the next kernel on this context
        __threadfence();
        const unsigned int prev = atomicAdd(&p.ctl->done, 1u);
        if (prev == gridDim.x - 1) {
            p.ctl->ticket = 0;
            p.ctl->done = 0;
        }
    }
}

int pow2_floor_g(int64_t v) {
    int q = 1;
    while ((int64_t)q * 2 <= v) q <<= 1;
    return q;
}

template <typename T>
const void* pick_grad_kernel(int ci) {
    switch (ci) {
        case 1: return (const void*)linear_grad_tma_kernel<T, 1>;
        case 2: return (const void*)linear_grad_tma_kernel<T, 2>;
        default: return (const void*)linear_grad_tma_kernel<T, 4>;
    }
}

}  // namespace

aa_status launch_assistant_grad_dense_tma(aa_ctx_impl* c, StepParams& p, int* parts_out) {
    const int es = p.f.dtype == AA_BF16 ? 2 : 4;
    const int ve = 16 / es;
    const int64_t row_bytes = p.f.d * es;
    if (row_bytes > kGMaxRowBytes || row_bytes < 1024) return AA_ERR_UNSUPPORTED;   // short rows: the load-based kernel
    if ((uintptr_t)p.f.w % 4) return AA_ERR_UNSUPPORTED;
    GradGeometry g;
    g.row_bytes = (uint32_t)row_bytes;
    g.nvec = (int)(p.f.d / ve);
    g.chunk_rows = pow2_floor_g(kGTargetStage / row_bytes);
    if (g.chunk_rows > 32) g.chunk_rows = 32;
    g.stage_bytes = (int)(((int64_t)g.chunk_rows * row_bytes + 127) / 128 * 128);
    g.split = g.chunk_rows >= 2 ? kDotSplit : 1;
    g.contiguous = (!p.row_idx && p.f.row_stride == p.f.d) ? 1 : 0;
    int ci = 1;
    while (ci < 4 && ci * kColThreads < g.nvec) ci <<= 1;
    if (ci * kColThreads < g.nvec) return AA_ERR_UNSUPPORTED;

    const size_t fixed = (size_t)p.f.d * sizeof(float) + sizeof(GradControl) + 128;
    const size_t budget = 220 * 1024;
    if (fixed + 2 * (size_t)g.stage_bytes > budget) return AA_ERR_UNSUPPORTED;
    int stages = (int)((budget - fixed) / g.stage_bytes);
    if (stages > kGMaxStages) stages = kGMaxStages;
    if (stages < kDotPairs) return AA_ERR_UNSUPPORTED;   // a dot pair must never be two ring passes behind
    g.stages = stages;
    const size_t smem = fixed + (size_t)stages * g.stage_bytes;

    const int64_t n_tickets = (p.m_host + kTicketRows - 1) / kTicketRows;
    int grid = c->sm_count;
    if (grid > n_tickets) grid = (int)n_tickets;
    if (grid < 1) grid = 1;
    if ((int64_t)grid * (p.d_pad + 1) > c->partial_floats) return AA_ERR_UNSUPPORTED;

    const void* kernel = p.f.dtype == AA_BF16 ? pick_grad_kernel<uint16_t>(ci) : pick_grad_kernel<float>(ci);
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return AA_ERR_CUDA;
    void* args[] = {&p, &g};
    if (cudaLaunchKernel(kernel, dim3(grid), dim3(kGradThreads), args, smem, c->stream) != cudaSuccess) return AA_ERR_CUDA;
    ++c->launches;
    *parts_out = grid;
    return AA_OK;
}

}  // namespace aa
