// Assistant gradient + update when the caller hands in the pre-activations that screening computed under the same
// parameters (sequential schedule: Algorithm 1 has just evaluated g(x_i; phi) for these instances, Algorithm 2's
// gradient needs the same values), for 16-byte aligned bf16 rows of up to 3072 features.  With nothing to multiply
// for the dot products, a batch row is read from shared memory once and no warp waits for another within a stage.
//
// A ring stage holds 8 batch rows (one bulk copy per row; rows padded by 16 bytes so that ldmatrix is
// bank-conflict free).  Column sums  sum_i r_i x_i  are  [16 features x 8 rows] x [8 rows x 8]  mma.m16n8k8 products
// whose left operand is the staged rows read transposed (ldmatrix.trans) and whose right operand carries r split
// into three bf16 terms (hi + mid + lo = all 24 bits of the fp32 residual) in three of its 8 columns.  bf16 x bf16
// products are exact in fp32 and the accumulators are fp32, so the arithmetic is that of an FMA loop up to
// summation order.
//
//   warp 0        producer: tickets of 16 batch rows (two stages), one bulk copy per row; publishes which rows a stage
//                 holds (a running stage count in shared memory) before its copies are issued.
//   warps 1, 2    the residuals r_i = sigmoid(score[row_i]) - z_i of a stage; the two warps take alternate
//                 stages (a stage's residuals hang on two dependent loads: batch list entry, then that row's score)
//                 and are done before the rows land.
//   warps 3..18   first the batch-mean threshold (all M losses, added in a fixed order in every CTA: no CTA waits for
//                 another), then column sums: each owns 12 feature blocks whose accumulator fragments stay in
//                 registers for the whole kernel.
// CTAs write column sums to the partial buffer; once all of them have (a cooperative launch keeps the grid
// co-resident, the wait is bounded all the same) each CTA adds up a slice of the columns and takes the SGD or Adam
// step for it, so the step is one launch.
#include <cuda_bf16.h>

#include "async_copy.cuh"
#include "step_common.cuh"

namespace aa {

namespace {

constexpr int kMRows = 8;                        // batch rows per ring stage
constexpr int kMMaxStages = 16;
constexpr int kResWarps = 2;                     // warps 1, 2: threshold and residuals
constexpr int kCompWarps = 16;                   // warps 3..18: dot products (one stage ahead) and column sums
constexpr int kMWarpsTotal = 1 + kResWarps + kCompWarps;
constexpr int kMThreads = kMWarpsTotal * 32;
constexpr int kMMaxBlocks = 12;                  // 16-feature blocks per compute warp: d <= 16 * 12 * 16 = 3072
constexpr int kMTicketRows = 16;                 // batch rows per ticket (two stages)

struct ScoredGeometry {
    int d;                // features (multiple of 16)
    int n_blocks;         // d / 16
    int stages;
    uint32_t row_bytes;   // d * 2
    uint32_t pitch;       // row_bytes + 16
    uint32_t stage_bytes; // kMRows * pitch rounded up to 128
    int contiguous;
};

struct ScoredControl {
    uint64_t x_full[kMMaxStages], x_empty[kMMaxStages];
    uint64_t r_ready[kMMaxStages];            // the stage's residuals are in r_split
    long long first_row[kMMaxStages];
    unsigned int valid[kMMaxStages];
    alignas(16) __nv_bfloat16 r_split[kMMaxStages][3][kMRows];   // hi / mid / lo terms of the residuals
    uint64_t t_ready;                         // every column warp's share of the loss sum is in t_part
    double t_part[kCompWarps];
    float bias_part[kResWarps];
    int published;                            // stage sequence numbers below this have their first_row / valid written
    int stop_j;
    int abort_flag;
};

__device__ __forceinline__ void scored_give_up(const StepParams& p, ScoredControl* cb) {
    latch(p.ctl, AA_ERR_SCAN_TIMEOUT);
    *(volatile int*)&cb->abort_flag = 1;
}

__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t& r0, uint32_t& r1, uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
// D += A (16x8, row) * B (8x8, col), bf16 operands, fp32 accumulation.
__device__ __forceinline__ void mma_bf16_1688(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5}, {%6}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(b0));
}

// Waits until the producer has published stage sequence number j (a running count in shared memory, not a barrier
// phase: with several residual warps each warp waits only for every few stages, and a phase parity cannot tell a stage
// from the one two ring passes later).  0 = published, 1 = the producer finished before reaching j, 2 = gave up.
__device__ __forceinline__ int wait_published(const volatile int* published, int j, const volatile int* stop_j, volatile int* abort_flag) {
    unsigned int polls = 0;
    while (true) {
        if (j >= *stop_j) return 1;
        if (*published > j) {
            __threadfence_block();
            return 0;
        }
        if (*abort_flag || ++polls > kSpinLimit) return 2;
        __nanosleep(polls < 16 ? 40 : 200);
    }
}

// v = hi + mid + lo with each term a bf16 (together the 24 significant bits of v).
__device__ __forceinline__ void split3(float v, __nv_bfloat16& hi, __nv_bfloat16& mid, __nv_bfloat16& lo) {
    hi = __float2bfloat16_rn(v);
    const float r1 = v - __bfloat162float(hi);
    mid = __float2bfloat16_rn(r1);
    lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
}

__global__ void __launch_bounds__(kMThreads, 1) linear_grad_scored_kernel(StepParams p, ScoredGeometry g) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* x_ring = smem;
    ScoredControl* cb = reinterpret_cast<ScoredControl*>(smem + (size_t)g.stages * g.stage_bytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int S = g.stages;
    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&cb->x_full[s], 1);
            mbar_init(&cb->x_empty[s], kCompWarps);
            mbar_init(&cb->r_ready[s], 1);
        }
        mbar_init(&cb->t_ready, kCompWarps);
        for (int q = 0; q < kResWarps; ++q) cb->bias_part[q] = 0.0f;
        cb->published = 0;
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
            if (tk >= n_tickets || lane >= kMTicketRows || i >= m) return -1;
            return g.contiguous ? (long long)i : batch_row(p, i);
        };
        // the first ticket of a CTA is its block index (no round trip before the first copies); the counter hands
        // out the tickets from gridDim.x on
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
                if (j >= S && !mbar_wait(&cb->x_empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                unsigned char* dst = x_ring + (size_t)stage * g.stage_bytes;
                const long long r = __shfl_sync(0xFFFFFFFFu, cur_row, (s * kMRows + lane) & 31);
                const bool mine = lane < kMRows && r >= 0;
                const unsigned int have = __ballot_sync(0xFFFFFFFFu, mine);
                if (lane == 0) {
                    cb->first_row[stage] = i0;
                    cb->valid[stage] = have;
                    __threadfence_block();
                    *(volatile int*)&cb->published = j + 1;
                    if (have) mbar_arrive_expect_tx(&cb->x_full[stage], (uint32_t)__popc(have) * g.row_bytes);
                    else mbar_arrive(&cb->x_full[stage]);
                }
                __syncwarp();
                if (mine) bulk_g2s(dst + (size_t)lane * g.pitch, base + (size_t)r * stride_bytes, g.row_bytes, &cb->x_full[stage]);
                __syncwarp();
                ++j;
                if (++stage == S) { stage = 0; phase ^= 1u; }
            }
            cur = next;
            cur_row = next_row;
            next = after;
        }
        if (ok) {
            // one empty stage wakes every other role for the last time
            if (j >= S && !mbar_wait(&cb->x_empty[stage], phase ^ 1u, abort_flag)) ok = false;
            if (ok && lane == 0) {
                *(volatile int*)&cb->stop_j = j;
                __threadfence_block();
                mbar_arrive(&cb->x_full[stage]);
            }
            ++j;
        }
        if (!ok) {
            if (lane == 0) scored_give_up(p, cb);
            const int pending = j < S ? j : S;
            for (int back = 1; back <= pending; ++back) {
                const int jj = j - back, st = jj % S, use = jj / S;
                const long long t0 = clock64();
                while (!mbar_try_wait(&cb->x_full[st], (uint32_t)(use & 1)) && clock64() - t0 < kWaitCycles) {}
            }
        }
    } else if (warp <= kResWarps) {
        const int aw = warp - 1;
        bool ok = true;
        // Shrinking threshold T: the caller's value, or the mean of the batch losses.  The sixteen column warps, which
        // have nothing to do until the first residuals exist, add all M losses in every CTA (a fixed order, so every CTA
        // and both residual warps arrive at the same bits); no CTA waits for another one.
        const bool mean_T = p.thresh_mode != AA_THRESH_VALUE;
        {
            // -------------------------------------------------------- residuals: the two warps take alternate stages
            const int n_res = kResWarps;
            double T_shrink = (double)p.threshold;
            bool have_T = !mean_T;
            float bias_acc = 0.0f;
            for (int j = aw; ok; j += n_res) {
                const int stage = j % S;
                const int pub = wait_published(&cb->published, j, &cb->stop_j, abort_flag);
                if (pub == 2) { ok = false; break; }
                if (pub == 1) break;
                const int64_t i0 = cb->first_row[stage];
                const unsigned int valid_rows = cb->valid[stage];
                const bool live = lane < kMRows && ((valid_rows >> lane) & 1u);
                float f_i = 0.0f, s_row = 0.0f;
                if (live) {
                    f_i = __ldg(p.loss + i0 + lane);
                    s_row = __ldg(p.score + (p.row_idx ? (int64_t)p.row_idx[i0 + lane] : i0 + lane));
                }
                if (!have_T) {
                    if (!mbar_wait(&cb->t_ready, 0, abort_flag)) { ok = false; break; }
                    double total = 0.0;
#pragma unroll
                    for (int q = 0; q < kCompWarps; ++q) total += *(volatile double*)&cb->t_part[q];
                    T_shrink = m > 0 ? total / (double)m : 0.0;
                    have_T = true;
                }
                if (lane < kMRows) {
                    float r = 0.0f;
                    if (live) {
                        const float z = (double)f_i > T_shrink ? 1.0f : 0.0f;
                        r = sigmoid_f32(s_row) - z;
                        bias_acc += r;
                    }
                    __nv_bfloat16 hi, mid, lo;
                    split3(r, hi, mid, lo);
                    cb->r_split[stage][0][lane] = hi;
                    cb->r_split[stage][1][lane] = mid;
                    cb->r_split[stage][2][lane] = lo;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&cb->r_ready[stage]);
            }
            if (!ok && lane == 0) scored_give_up(p, cb);
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) bias_acc += __shfl_xor_sync(0xFFFFFFFFu, bias_acc, o);
            if (lane == 0) cb->bias_part[aw] = bias_acc;
        }
    } else {
        // ------------------------------------------------------------ column sums
        const int cw = warp - (1 + kResWarps);
        const int gid = lane >> 2, tq = lane & 3;     // fragment coordinates of this lane
        float acc[kMMaxBlocks][4];                    // [feature block of this warp][fragment]: sum_i r_i x_i (three terms side by side)
#pragma unroll
        for (int q = 0; q < kMMaxBlocks; ++q)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[q][e] = 0.0f;
        if (p.thresh_mode != AA_THRESH_VALUE) {
            // this warp's share of the loss sum: elements (or 16-byte groups) cw * 32 + lane, + 512, ...; then a shuffle tree
            const int ct = cw * 32 + lane;
            double part = 0.0;
            if (((uintptr_t)p.loss & 15) == 0) {
                const int64_t quads = m >> 2;
                const float4* l4 = reinterpret_cast<const float4*>(p.loss);
                int64_t q = ct;
                for (; q + 3 * kCompWarps * 32 < quads; q += 4 * kCompWarps * 32) {        // four loads in flight together
                    const float4 a = __ldg(l4 + q), b = __ldg(l4 + q + kCompWarps * 32), c4 = __ldg(l4 + q + 2 * kCompWarps * 32),
                                 d4 = __ldg(l4 + q + 3 * kCompWarps * 32);
                    part += ((double)a.x + (double)a.y) + ((double)a.z + (double)a.w);
                    part += ((double)b.x + (double)b.y) + ((double)b.z + (double)b.w);
                    part += ((double)c4.x + (double)c4.y) + ((double)c4.z + (double)c4.w);
                    part += ((double)d4.x + (double)d4.y) + ((double)d4.z + (double)d4.w);
                }
                for (; q < quads; q += kCompWarps * 32) {
                    const float4 a = __ldg(l4 + q);
                    part += ((double)a.x + (double)a.y) + ((double)a.z + (double)a.w);
                }
                for (int64_t i = (quads << 2) + ct; i < m; i += kCompWarps * 32) part += (double)__ldg(p.loss + i);
            } else {
                for (int64_t i = ct; i < m; i += kCompWarps * 32) part += (double)__ldg(p.loss + i);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, o);
            if (lane == 0) {
                cb->t_part[cw] = part;
                mbar_arrive(&cb->t_ready);
            }
            __syncwarp();
        }
        bool ok = true;
        for (int j = 0; ok; ++j) {
            const int stage = j % S, use = j / S;
            if (!mbar_wait(&cb->x_full[stage], (uint32_t)(use & 1), abort_flag)) {
                if (lane == 0) scored_give_up(p, cb);
                break;
            }
            if (j >= *(volatile int*)&cb->stop_j) break;
            if (!mbar_wait(&cb->r_ready[stage], (uint32_t)(use & 1), abort_flag)) {
                if (lane == 0) scored_give_up(p, cb);
                break;
            }
            const unsigned int valid_rows = cb->valid[stage];
            const uint32_t xs = smem_u32(x_ring + (size_t)stage * g.stage_bytes);
            const int first_valid = valid_rows ? __ffs(valid_rows) - 1 : 0;
            const int my_row = lane & 7;
            const int t_row = ((valid_rows >> my_row) & 1u) ? my_row : first_valid;
            const uint32_t t_base = xs + (uint32_t)t_row * g.pitch + (uint32_t)(((lane >> 3) & 1) * 16);
            uint32_t rb0 = 0;                          // right operand: rows 2tq, 2tq + 1 of term gid
            if (gid < 3) rb0 = *reinterpret_cast<const uint32_t*>(&cb->r_split[stage][gid][2 * tq]);
#pragma unroll
            for (int q = 0; q < kMMaxBlocks; ++q) {
                const int kb = cw + q * kCompWarps;
                if (kb < g.n_blocks && valid_rows) {      // (a stage none of whose rows could be fetched holds only stale bytes)
                    uint32_t a0, a1;      // features 0..7 and 8..15 of the block x the stage's 8 rows
                    ldmatrix_x2_trans(a0, a1, t_base + (uint32_t)kb * 32);
                    mma_bf16_1688(acc[q], a0, a1, rb0);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&cb->x_empty[stage]);
        }
        // this CTA's column sums: feature kb*16 + gid (+8) = the three terms added up
        float* part = p.partials + (int64_t)blockIdx.x * p.d_pad;
#pragma unroll
        for (int q = 0; q < kMMaxBlocks; ++q) {
            const int kb = cw + q * kCompWarps;
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
        float bias_sum = 0.0f;
        for (int q = 0; q < kResWarps; ++q) bias_sum += cb->bias_part[q];
        p.partials[(int64_t)gridDim.x * p.d_pad + blockIdx.x] = bias_sum;
        __threadfence();
        atomicAdd(&p.ctl->grad_done, 1u);
        unsigned int polls = 0;
        while (*(volatile unsigned int*)&p.ctl->grad_done < gridDim.x && !*abort_flag) {
            if (++polls > kSpinLimit) break;
            __nanosleep(64);
        }
        if (*(volatile unsigned int*)&p.ctl->grad_done < gridDim.x || *abort_flag) {
            scored_give_up(p, cb);
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
                float part_v[8];   // 148 CTAs over 19 warps: at most 8 partials per lane, all loads in flight together
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const unsigned int q = warp + u * kAllWarps;
                    part_v[u] = q < gridDim.x ? __ldcg(p.partials + (int64_t)q * p.d_pad + jcol) : 0.0f;
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) gsum += part_v[u];
                for (unsigned int q = warp + 8 * kAllWarps; q < gridDim.x; q += kAllWarps) gsum += __ldcg(p.partials + (int64_t)q * p.d_pad + jcol);
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

aa_status launch_assistant_grad_dense_scored(aa_ctx_impl* c, StepParams& p, int* parts_out) {
    if (!p.score || p.f.dtype != AA_BF16 || p.f.d % 16 || p.f.d < 256 || p.f.d > kCompWarps * kMMaxBlocks * 16) return AA_ERR_UNSUPPORTED;
    if ((uintptr_t)p.f.base % 16 || (p.f.row_stride * 2) % 16 || (uintptr_t)p.f.w % 4) return AA_ERR_UNSUPPORTED;
    ScoredGeometry g;
    g.d = (int)p.f.d;
    g.n_blocks = g.d / 16;
    g.row_bytes = (uint32_t)g.d * 2u;
    g.pitch = g.row_bytes + 16u;
    g.stage_bytes = ((uint32_t)kMRows * g.pitch + 127u) & ~127u;
    g.contiguous = (!p.row_idx && p.f.row_stride == p.f.d) ? 1 : 0;
    const size_t fixed = sizeof(ScoredControl) + 128;
    const size_t budget = 222 * 1024;
    if (fixed + 2 * (size_t)g.stage_bytes > budget) return AA_ERR_UNSUPPORTED;
    int stages = (int)((budget - fixed) / g.stage_bytes);
    g.stages = stages > kMMaxStages ? kMMaxStages : stages;
    const size_t smem = (size_t)g.stages * g.stage_bytes + fixed;
    const int64_t n_tickets = (p.m_host + kMTicketRows - 1) / kMTicketRows;
    int grid = c->sm_count;
    if (grid > n_tickets) grid = (int)n_tickets;
    if (grid < 1) grid = 1;
    // partial buffer: [grid][d_pad] column sums, then [grid] bias sums
    if ((int64_t)grid * (p.d_pad + 1) > c->partial_floats) return AA_ERR_UNSUPPORTED;
    p.loss_sums = nullptr;
    const void* kernel = (const void*)linear_grad_scored_kernel;
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
