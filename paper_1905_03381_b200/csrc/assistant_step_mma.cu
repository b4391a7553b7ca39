// Assistant gradient for 16-byte aligned bf16 rows of up to 3072 features (Sec. "Learning to generate smart training batches" objective;
// Algorithm 2: Assistant.gradient), with the two passes over each staged row done by warp-level
// matrix instructions instead of one FMA per element.
//
// The pass over a batch row costs the load-based and bulk-copy kernels about four scalar
// instructions per feature (unpack + FMA for the dot product, unpack + FMA for r * x), which makes
// them issue-bound before they are bandwidth-bound.  Here a ring stage holds 16 rows and
//   dot products   s_i = w . x_i   are   [16 rows x 16 features] x [16 features x 8] mma.m16n8k16
//                  products whose right operand carries w split into three bf16 terms
//                  (hi + mid + lo = all 24 bits of the fp32 weight) in three of its 8 columns;
//   column sums    sum_i r_i x_i   are   [16 features x 16 rows] x [16 rows x 8]  products whose left
//                  operand is the staged rows read transposed (ldmatrix.trans) and whose right
//                  operand carries r split the same way.
// bf16 x bf16 products are exact in fp32 and the accumulators are fp32, so the arithmetic is that of
// the FMA kernels up to summation order.  One ldmatrix + one mma handle 256 features of 16 rows.
//
//   producer warp  : tickets of 16 batch rows, one bulk copy per row into a 2-stage ring (rows
//                    padded by 16 bytes so that ldmatrix is bank-conflict free), the stage's losses
//                    ride along.
//   12 compute warps: each takes a share of the feature blocks for the dot products, the shares
//                    meet in shared memory (mbarrier, bounded wait), every warp forms the 16
//                    residuals r = sigmoid(s) - z, then adds r * x for its own 256 columns into
//                    accumulator fragments that live in registers for the whole kernel.
// CTAs write column sums to the partial buffer; once all of them have (a cooperative launch keeps the
// grid co-resident, the wait is bounded all the same) each CTA adds up a slice of the columns and
// takes the SGD or Adam step for it, so the step is one launch.
#include <cuda_bf16.h>

#include "async_copy.cuh"
#include "step_common.cuh"

namespace aa {

namespace {

constexpr int kFragRows = 16;                    // rows of one matrix-instruction operand
constexpr int kMRows = 16;                       // batch rows per ring stage
constexpr int kMStages = 2;
constexpr int kMWarps = 12;                      // compute warps
constexpr int kMThreads = (1 + kMWarps) * 32;
constexpr int kMMaxBlocks = 16;                  // 16-feature blocks per warp: d <= 12 * 16 * 16 = 3072
constexpr int kMTicketRows = 16;                 // batch rows per ticket: one ring stage (8-row stages measured 2x slower:
                                                 // the per-stage exchange and residuals are paid by every warp)

struct MmaGeometry {
    int d;                // features (multiple of 16)
    int n_blocks;         // d / 16
    uint32_t row_bytes;   // d * 2
    uint32_t pitch;       // row_bytes + 16
    uint32_t stage_bytes; // kMRows * pitch rounded up to 128
    int contiguous;
};

struct MmaControl {
    uint64_t x_full[kMStages], x_empty[kMStages], dots_in[kMStages];
    uint64_t t_ready;                         // the batch-mean threshold is in T_mean (posted by the producer warp)
    long long first_row[kMStages];
    unsigned int valid[kMStages];
    alignas(16) float loss[kMStages][kMRows];
    int loss_staged[kMStages];
    float part[kMStages][kMWarps][kFragRows];     // each warp's share of the dot products
    alignas(4) __nv_bfloat16 r_split[kMWarps][3][kFragRows];   // per warp: hi / mid / lo terms of the residuals
    double red[kMWarps];
    double T_mean;
    float bias_sum;
    int stop_j;
    int abort_flag;
};

__device__ __forceinline__ void mma_give_up(const StepParams& p, MmaControl* cb) {
    latch(p.ctl, AA_ERR_SCAN_TIMEOUT);
    *(volatile int*)&cb->abort_flag = 1;
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D += A (16x16, row) * B (16x8, col), bf16 operands, fp32 accumulation.
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// v = hi + mid + lo with each term a bf16 (together the 24 significant bits of v).
__device__ __forceinline__ void split3(float v, __nv_bfloat16& hi, __nv_bfloat16& mid, __nv_bfloat16& lo) {
    hi = __float2bfloat16_rn(v);
    const float r1 = v - __bfloat162float(hi);
    mid = __float2bfloat16_rn(r1);
    lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
}

__global__ void __launch_bounds__(kMThreads, 1) linear_grad_mma_kernel(StepParams p, MmaGeometry g) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* x_ring = smem;
    // w as three bf16 planes: w_split[term][feature]
    __nv_bfloat16* w_split = reinterpret_cast<__nv_bfloat16*>(smem + (size_t)kMStages * g.stage_bytes);
    MmaControl* cb = reinterpret_cast<MmaControl*>(reinterpret_cast<unsigned char*>(w_split) + (((size_t)3 * g.d * 2 + 127) & ~(size_t)127));

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kMStages; ++s) {
            mbar_init(&cb->x_full[s], 1);
            mbar_init(&cb->x_empty[s], kMWarps);
            mbar_init(&cb->dots_in[s], kMWarps);
        }
        mbar_init(&cb->t_ready, 1);
        cb->bias_sum = 0.0f;
        cb->stop_j = 0x7FFFFFFF;
        cb->abort_flag = 0;
        mbar_fence_init();
    }
    volatile int* abort_flag = &cb->abort_flag;
    __syncthreads();   // barriers are initialised
    // everything above overlapped the previous kernel's tail; from here on its results are read (batch, losses, counters)
    grid_dependency_wait();
    grid_dependency_release();
    const int64_t m = batch_size(p);

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        const unsigned char* base = static_cast<const unsigned char*>(p.f.base);
        const size_t stride_bytes = (size_t)p.f.row_stride * 2;
        const unsigned int n_tickets = (unsigned int)((m + kMTicketRows - 1) / kMTicketRows);
        int j = 0, stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        auto fetch_row = [&](unsigned int tk) -> long long {
            const int64_t i = (int64_t)tk * kMTicketRows + lane;
            if (tk >= n_tickets || i >= m) return -1;
            return g.contiguous ? (long long)i : batch_row(p, i);
        };
        // the first ticket of a CTA is its block index (no round trip before the first copies); the counter hands
        // out the tickets from gridDim.x on
        // The batch-mean threshold: once the ring is full (or the batch has run out) this warp, idle until a stage is
        // released, waits for every CTA's share of the loss sum, adds them in CTA order and posts the mean.
        bool t_posted = p.thresh_mode == AA_THRESH_VALUE;
        auto post_threshold = [&]() {
            unsigned int polls = 0;
            while (*(volatile unsigned int*)&p.ctl->sums_in < gridDim.x && !*abort_flag) {
                if (++polls > kSpinLimit) break;
                __nanosleep(32);
            }
            if (*(volatile unsigned int*)&p.ctl->sums_in < gridDim.x) {
                if (lane == 0) mma_give_up(p, cb);
            } else {
                __threadfence();
                double share[5];      // lane l adds shares l, l + 32, ... (loads in flight together); then a fixed shuffle tree
#pragma unroll
                for (int u = 0; u < 5; ++u) share[u] = lane + 32u * u < gridDim.x ? __ldcg(p.loss_sums + lane + 32 * u) : 0.0;
                double total = 0.0;
#pragma unroll
                for (int u = 0; u < 5; ++u) total += share[u];
                for (unsigned int q = lane + 160; q < gridDim.x; q += 32) total += __ldcg(p.loss_sums + q);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xFFFFFFFFu, total, o);
                if (lane == 0) {
                    cb->T_mean = m > 0 ? total / (double)m : 0.0;
                    mbar_arrive(&cb->t_ready);
                }
            }
            t_posted = true;
        };
        unsigned int cur = blockIdx.x, next = 0;
        long long cur_row = fetch_row(cur);
        if (lane == 0) next = gridDim.x + atomicAdd(&p.ctl->ticket, 1u);
        while (ok && cur < n_tickets) {
            next = __shfl_sync(0xFFFFFFFFu, next, 0);
            const long long next_row = fetch_row(next);       // on its way while this ticket is issued
            unsigned int after = 0;
            if (lane == 0) after = gridDim.x + atomicAdd(&p.ctl->ticket, 1u);
            for (int s = 0; s < kMTicketRows / kMRows; ++s) {
                const int64_t i0 = (int64_t)cur * kMTicketRows + (int64_t)s * kMRows;
                if (i0 >= m) break;
                if (j >= kMStages && !t_posted) post_threshold();
                if (j >= kMStages && !mbar_wait(&cb->x_empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                unsigned char* dst = x_ring + (size_t)stage * g.stage_bytes;
                const long long r = __shfl_sync(0xFFFFFFFFu, cur_row, (s * kMRows + lane) & 31);
                const bool mine = lane < kMRows && r >= 0;
                const unsigned int have = __ballot_sync(0xFFFFFFFFu, mine);
                const uint32_t loss_bytes = (__popc(have) == kMRows && i0 + kMRows <= m && (((uintptr_t)(p.loss + i0)) & 15) == 0)
                                                ? (uint32_t)kMRows * 4u : 0u;
                if (lane == 0) {
                    cb->first_row[stage] = i0;
                    cb->valid[stage] = have;
                    cb->loss_staged[stage] = loss_bytes != 0;
                    if (have) mbar_arrive_expect_tx(&cb->x_full[stage], (uint32_t)__popc(have) * g.row_bytes + loss_bytes);
                    else mbar_arrive(&cb->x_full[stage]);
                    if (loss_bytes) bulk_g2s(&cb->loss[stage][0], p.loss + i0, loss_bytes, &cb->x_full[stage]);
                }
                __syncwarp();
                if (mine) bulk_g2s(dst + (size_t)lane * g.pitch, base + (size_t)r * stride_bytes, g.row_bytes, &cb->x_full[stage]);
                __syncwarp();
                ++j;
                if (++stage == kMStages) { stage = 0; phase ^= 1u; }
            }
            cur = next;
            cur_row = next_row;
            next = after;
        }
        if (!t_posted) post_threshold();
        if (ok) {
            // one empty stage wakes the compute warps for the last time
            if (lane == 0) *(volatile int*)&cb->stop_j = j;
            if (j >= kMStages && !mbar_wait(&cb->x_empty[stage], phase ^ 1u, abort_flag)) ok = false;
            if (ok && lane == 0) mbar_arrive(&cb->x_full[stage]);
            ++j;
        }
        if (!ok) {
            if (lane == 0) mma_give_up(p, cb);
            const int pending = j < kMStages ? j : kMStages;
            for (int back = 1; back <= pending; ++back) {
                const int jj = j - back, st = jj % kMStages, use = jj / kMStages;
                const long long t0 = clock64();
                while (!mbar_try_wait(&cb->x_full[st], (uint32_t)(use & 1)) && clock64() - t0 < kWaitCycles) {}
            }
        }
    } else {
        // ------------------------------------------------------------ compute warps
        const int cw = warp - 1;
        const int ct = tid - 32;
        // weights as three bf16 planes, and the batch-mean threshold (fixed order: thread stride, warp tree, warp index)
        const bool mean_T = p.thresh_mode != AA_THRESH_VALUE;
        // this CTA's slice of the losses (batch-mean threshold): the first load is issued ahead of the weight loads
        const int64_t per = ((m + gridDim.x - 1) / gridDim.x + 3) / 4 * 4;
        const int64_t s_lo = (int64_t)blockIdx.x * per, s_hi = s_lo + per < m ? s_lo + per : m;
        const float first_loss = (mean_T && s_lo + ct < s_hi) ? __ldg(p.loss + s_lo + ct) : 0.0f;
        for (int jf = ct; jf < g.d; jf += kMWarps * 32) {
            __nv_bfloat16 hi, mid, lo;
            split3(__ldcg(p.f.w + jf), hi, mid, lo);       // w is rewritten at the end of this kernel: no read-only path
            w_split[jf] = hi;
            w_split[g.d + jf] = mid;
            w_split[2 * g.d + jf] = lo;
        }
        // Batch-mean threshold: summing all M losses in every CTA costs more than the first ring stage, so each CTA adds
        // one slice (fixed order: thread stride, warp tree, warp index), publishes its share, and all CTAs add the shares
        // in one fixed order once everyone has published (the producer warp does that while the ring is full).
        double T_shrink = (double)p.threshold;
        if (mean_T) {
            double acc = (double)first_loss;
            for (int64_t i = s_lo + ct + kMWarps * 32; i < s_hi; i += kMWarps * 32) acc += (double)__ldg(p.loss + i);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
            if (lane == 0) cb->red[cw] = acc;
        }
        asm volatile("bar.sync 2, %0;" ::"n"(kMWarps * 32) : "memory");
        if (mean_T && ct == 0) {
            double total = 0.0;
            for (int wi = 0; wi < kMWarps; ++wi) total += cb->red[wi];
            p.loss_sums[blockIdx.x] = total;
            __threadfence();
            atomicAdd(&p.ctl->sums_in, 1u);
        }
        bool have_T = !mean_T;
        const float bias = *p.f.b;
        const int gid = lane >> 2, tq = lane & 3;     // fragment coordinates of this lane
        float acc[kMMaxBlocks][4];                    // [feature block of this warp][fragment]: sum_i r_i x_i (three terms side by side)
#pragma unroll
        for (int q = 0; q < kMMaxBlocks; ++q)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[q][e] = 0.0f;
        float bias_acc = 0.0f;

        for (int j = 0;; ++j) {
            const int stage = j % kMStages, use = j / kMStages;
            if (!mbar_wait(&cb->x_full[stage], (uint32_t)(use & 1), abort_flag)) {
                if (lane == 0) mma_give_up(p, cb);
                break;
            }
            if (j >= *(volatile int*)&cb->stop_j) break;
            const int64_t i0 = cb->first_row[stage];
            const unsigned int valid_rows = cb->valid[stage];
            const uint32_t xs = smem_u32(x_ring + (size_t)stage * g.stage_bytes);
            // Rows that were not fetched hold stale bytes: every matrix load reads a fetched row in their place
            // (their dot products are ignored and their residuals are zero).
            const int first_valid = __ffs(valid_rows) - 1;
            auto safe_row = [&](int r) { return ((valid_rows >> r) & 1u) ? r : first_valid; };

            // ---- dot products: this warp's feature blocks
            float dot[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            {
                float dot2[4] = {0.0f, 0.0f, 0.0f, 0.0f};       // two accumulators: consecutive products do not wait on each other
                const int a_row = safe_row((lane & 7) + ((lane >> 3) & 1) * 8);
                const uint32_t a_base = xs + (uint32_t)a_row * g.pitch + (uint32_t)((lane >> 4) * 16);
                int flip = 0;
                for (int kb = cw; kb < g.n_blocks; kb += kMWarps, flip ^= 1) {
                    uint32_t a[4];
                    ldmatrix_x4(a, a_base + (uint32_t)kb * 32);
                    uint32_t b0 = 0, b1 = 0;
                    if (gid < 3) {
                        const __nv_bfloat16* wp = w_split + (size_t)gid * g.d + kb * 16 + 2 * tq;
                        b0 = *reinterpret_cast<const uint32_t*>(wp);
                        b1 = *reinterpret_cast<const uint32_t*>(wp + 8);
                    }
                    if (flip) mma_bf16_16816(dot2, a, b0, b1);
                    else mma_bf16_16816(dot, a, b0, b1);
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) dot[e] += dot2[e];
            }
            // columns 0..2 of the product hold the three terms: lanes tq = 0 (columns 0, 1) and tq = 1 (column 2)
            float lo_row = dot[0] + dot[1], hi_row = dot[2] + dot[3];       // rows gid and gid + 8
            lo_row += __shfl_xor_sync(0xFFFFFFFFu, lo_row, 1);
            hi_row += __shfl_xor_sync(0xFFFFFFFFu, hi_row, 1);
            if (tq == 0) {
                cb->part[stage][cw][gid] = lo_row;
                cb->part[stage][cw][gid + 8] = hi_row;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&cb->dots_in[stage]);
            if (!mbar_wait(&cb->dots_in[stage], (uint32_t)(use & 1), abort_flag)) {
                if (lane == 0) mma_give_up(p, cb);
                break;
            }
            if (!have_T) {
                // the producer warp posts the mean once every CTA's share is in
                if (!mbar_wait(&cb->t_ready, 0, abort_flag)) {
                    if (lane == 0) mma_give_up(p, cb);
                    break;
                }
                T_shrink = *(volatile double*)&cb->T_mean;
                have_T = true;
            }
            // ---- residuals of the 16 rows (every warp, lanes 0..15), split into three bf16 terms
            if (lane < kFragRows) {
                float r = 0.0f;
                if ((valid_rows >> lane) & 1u) {
                    float s_row = bias;
#pragma unroll
                    for (int w = 0; w < kMWarps; ++w) s_row += cb->part[stage][w][lane];
                    const float f_i = cb->loss_staged[stage] ? cb->loss[stage][lane] : __ldg(p.loss + i0 + lane);
                    const float z = (double)f_i > T_shrink ? 1.0f : 0.0f;
                    r = sigmoid_f32(s_row) - z;
                    if (cw == 0) bias_acc += r;
                }
                __nv_bfloat16 hi, mid, lo;
                split3(r, hi, mid, lo);
                cb->r_split[cw][0][lane] = hi;
                cb->r_split[cw][1][lane] = mid;
                cb->r_split[cw][2][lane] = lo;
            }
            __syncwarp();
            uint32_t rb0 = 0, rb1 = 0;                // right operand: rows 2tq, 2tq+1 (and +8) of term gid
            if (gid < 3) {
                rb0 = *reinterpret_cast<const uint32_t*>(&cb->r_split[cw][gid][2 * tq]);
                rb1 = *reinterpret_cast<const uint32_t*>(&cb->r_split[cw][gid][2 * tq + 8]);
            }
            // ---- column sums: this warp's feature blocks, rows read transposed
            {
                const int t_row = safe_row((lane & 7) + (lane >> 4) * 8);
                const uint32_t t_base = xs + (uint32_t)t_row * g.pitch + (uint32_t)(((lane >> 3) & 1) * 16);
#pragma unroll
                for (int q = 0; q < kMMaxBlocks; ++q) {
                    const int kb = cw + q * kMWarps;
                    if (kb < g.n_blocks) {
                        uint32_t a[4];
                        ldmatrix_x4_trans(a, t_base + (uint32_t)kb * 32);
                        mma_bf16_16816(acc[q], a, rb0, rb1);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&cb->x_empty[stage]);
        }
        // this CTA's column sums: feature kb*16 + gid (+8) = the three terms added up
        float* part = p.partials + (int64_t)blockIdx.x * p.d_pad;
#pragma unroll
        for (int q = 0; q < kMMaxBlocks; ++q) {
            const int kb = cw + q * kMWarps;
            if (kb < g.n_blocks) {
                float lo_col = acc[q][0] + acc[q][1], hi_col = acc[q][2] + acc[q][3];
                lo_col += __shfl_xor_sync(0xFFFFFFFFu, lo_col, 1);
                hi_col += __shfl_xor_sync(0xFFFFFFFFu, hi_col, 1);
                if (tq == 0) {
                    part[kb * 16 + gid] = lo_col;
                    part[kb * 16 + gid + 8] = hi_col;
                }
            }
        }
        if (cw == 0) {
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) bias_acc += __shfl_xor_sync(0xFFFFFFFFu, bias_acc, o);
            if (lane == 0) cb->bias_sum = bias_acc;
        }
    }
    // the weights this CTA will update are read while the partial sums of the other CTAs are still on their way
    const int cols_per_cta = (g.d + (int)gridDim.x - 1) / (int)gridDim.x;
    const int c0 = (int)blockIdx.x * cols_per_cta;
    const int c1 = c0 + cols_per_cta < g.d ? c0 + cols_per_cta : g.d;
    float w_first = 0.0f;
    if (warp == 0 && c0 + lane < c1) w_first = __ldcg(p.w + c0 + lane);
    __syncthreads();
    // ---------------------------------------------------------------- update (Algorithm 2: Assistant.update)
    // Every CTA publishes its sums, waits (bounded) until all CTAs of this cooperative launch have done so, then adds
    // the partial sums of its own slice of the columns in a fixed order and takes the step for that slice.
    if (tid == 0) {
        p.partials[(int64_t)gridDim.x * p.d_pad + blockIdx.x] = cb->bias_sum;
        __threadfence();
        atomicAdd(&p.ctl->grad_done, 1u);
        unsigned int polls = 0;
        while (*(volatile unsigned int*)&p.ctl->grad_done < gridDim.x && !*abort_flag) {
            if (++polls > kSpinLimit) break;
            __nanosleep(64);
        }
        if (*(volatile unsigned int*)&p.ctl->grad_done < gridDim.x || *abort_flag) {
            mma_give_up(p, cb);
        } else {
            __threadfence();
            // the last CTA past the wait re-arms the counters for the next kernel on this context
            const unsigned int prev = atomicAdd(&p.ctl->applied, 1u);
            if (prev == gridDim.x - 1) {
                p.ctl->ticket = 0;
                p.ctl->grad_done = 0;
                p.ctl->sums_in = 0;
                p.ctl->applied = 0;
            }
        }
    }
    __syncthreads();
    if (*abort_flag || m <= 0) return;
    {
        float* share = reinterpret_cast<float*>(x_ring);            // [warps][32]; every copy into the ring has landed
        constexpr int kAllWarps = kMThreads / 32;
        const float scale = p.lr / (float)m;
        for (int cb0 = c0; cb0 < c1; cb0 += 32) {
            const int jcol = cb0 + lane;
            float gsum = 0.0f;
            if (jcol < c1) {
                float part_v[12];   // 148 CTAs over 13 warps: at most 12 partials per lane, all loads in flight together
#pragma unroll
                for (int u = 0; u < 12; ++u) {
                    const unsigned int q = warp + u * kAllWarps;
                    part_v[u] = q < gridDim.x ? __ldcg(p.partials + (int64_t)q * p.d_pad + jcol) : 0.0f;
                }
#pragma unroll
                for (int u = 0; u < 12; ++u) gsum += part_v[u];
                for (unsigned int q = warp + 12 * kAllWarps; q < gridDim.x; q += kAllWarps) gsum += __ldcg(p.partials + (int64_t)q * p.d_pad + jcol);
            }
            share[warp * 32 + lane] = gsum;
            __syncthreads();
            if (warp == 0 && jcol < c1) {
                float t = 0.0f;
#pragma unroll
                for (int k = 0; k < kAllWarps; ++k) t += share[k * 32 + lane];
                const float w_old = cb0 == c0 ? w_first : __ldcg(p.w + jcol);
                p.w[jcol] = p.adam.on ? adam_update(p.adam, w_old, t / (float)m, p.lr, jcol) : w_old - scale * t;
            }
            __syncthreads();
        }
        if (blockIdx.x == 0 && warp == 1) {
            float t = 0.0f;
            for (unsigned int q = lane; q < gridDim.x; q += 32) t += __ldcg(p.partials + (int64_t)gridDim.x * p.d_pad + q);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
            if (lane == 0) p.b[0] = p.adam.on ? adam_update(p.adam, p.b[0], t / (float)m, p.lr, p.f.d) : p.b[0] - scale * t;
        }
    }
}

}  // namespace

aa_status launch_assistant_grad_dense_mma(aa_ctx_impl* c, StepParams& p, int* parts_out) {
    if (p.f.dtype != AA_BF16 || p.f.d % 16 || p.f.d < 256 || p.f.d > kMWarps * kMMaxBlocks * 16) return AA_ERR_UNSUPPORTED;
    if ((uintptr_t)p.f.base % 16 || (p.f.row_stride * 2) % 16 || (uintptr_t)p.f.w % 4) return AA_ERR_UNSUPPORTED;
    MmaGeometry g;
    g.d = (int)p.f.d;
    g.n_blocks = g.d / 16;
    g.row_bytes = (uint32_t)g.d * 2u;
    g.pitch = g.row_bytes + 16u;
    g.stage_bytes = ((uint32_t)kMRows * g.pitch + 127u) & ~127u;
    g.contiguous = (!p.row_idx && p.f.row_stride == p.f.d) ? 1 : 0;
    const size_t smem = (size_t)kMStages * g.stage_bytes + (((size_t)3 * g.d * 2 + 127) & ~(size_t)127) + sizeof(MmaControl) + 128;
    if (smem > 225 * 1024) return AA_ERR_UNSUPPORTED;
    const int64_t n_tickets = (p.m_host + kMTicketRows - 1) / kMTicketRows;
    int grid = c->sm_count;
    if (grid > n_tickets) grid = (int)n_tickets;
    if (grid < 1) grid = 1;
    // partial buffer: [grid][d_pad] column sums, [grid] bias sums, then [grid] doubles for the shares of the loss sum
    const int64_t sums_at = ((int64_t)grid * (p.d_pad + 1) + 1) / 2 * 2;
    if (sums_at + 2 * (int64_t)grid > c->partial_floats) return AA_ERR_UNSUPPORTED;
    p.loss_sums = reinterpret_cast<double*>(c->partials + sums_at);
    const void* kernel = (const void*)linear_grad_mma_kernel;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return AA_ERR_CUDA;
    void* args[] = {&p, &g};
    // cooperative: the CTAs wait for one another before the update, so all of them must be resident at once
    const cudaError_t le = launch_overlapped(c, kernel, dim3(grid), dim3(kMThreads), args, smem, true);
    if (le == cudaErrorCooperativeLaunchTooLarge || le == cudaErrorNotSupported) {
        // the device cannot hold the whole grid at once (or has no cooperative launch): the other gradient kernels wait on nobody
        (void)cudaGetLastError();
        return AA_ERR_UNSUPPORTED;
    }
    if (le != cudaSuccess) return AA_ERR_CUDA;
    ++c->launches;
    *parts_out = 0;   // the update was taken inside the kernel
    return AA_OK;
}

}  // namespace aa
