// Per-instance Boss loss (Sec. 5.3) for 16-byte aligned logit rows of up to 16 KB, as one persistent,
// warp-specialised CTA per SM fed by bulk asynchronous copies.
//
// The logit matrix is cut into units of 2..32 whole rows (about 24 KB); units are handed out by a
// ticket counter (four at a time), so the CTAs stay balanced.
//   producer warp : takes tickets and streams each unit into a shared-memory ring with
//                   cp.async.bulk; the unit's labels ride along when their slice is aligned.
//   consumer warps: two per ring stage.  LPR lanes per row keep a running (max, sum) of the
//                   one-pass log-sum-exp, merge by shuffles and write the row's loss (the label's
//                   logit is read from the staged row).
// Longer rows, unaligned rows and small problems use the load-based kernels of instance_loss.cu,
// which measured as fast or faster there.
// Every wait is bounded; a role that gives up latches AA_ERR_SCAN_TIMEOUT and all roles drain.
#include "async_copy.cuh"
#include "loss_common.cuh"

namespace aa {

namespace {

constexpr int kLMaxStages = 8;
constexpr int kLSplit = 2;                                   // consumer warps per stage
constexpr int kLConsumers = kLMaxStages * kLSplit;
constexpr int kLossThreads = (1 + kLConsumers) * 32;         // warp 0 producer, 1..16 consumers
constexpr int kLTargetStage = 24 * 1024;
constexpr int kUnitsPerTicket = 4;
constexpr int64_t kMinRingBytes = 128ll << 20;               // below this the launch-light kernels win

struct LossGeometry {
    int chunk_rows;         // rows per unit (power of two, 2..32)
    uint32_t row_bytes;
    int stage_bytes;
    int stages;
    int contiguous;         // the rows of a unit are adjacent in memory
    int nvec;               // 16-byte vectors per row
};

struct LossRing {
    uint64_t full[kLMaxStages], empty[kLMaxStages];
    long long unit_of_stage[kLMaxStages];
    alignas(16) int labels[kLMaxStages][32];   // the unit's labels, when labels_staged[stage] is set
    int labels_staged[kLMaxStages];
    int stop_j;
    int abort_flag;
};

__device__ __forceinline__ void loss_give_up(const LossParams& p, LossRing* cb) {
    latch(p.ctl, AA_ERR_SCAN_TIMEOUT);
    *(volatile int*)&cb->abort_flag = 1;
}

// Short rows: `rows` staged rows of this warp, LPR lanes per row, first row is global row r0.
template <typename T, int LPR>
__device__ __forceinline__ void consume_short(const LossParams& p, const LossGeometry& g, const unsigned char* xs, int rows,
                                              int64_t r0, int64_t n_rows, const int* lab_s, int lane) {
    constexpr int VE = Vec<T>::kElems;
    constexpr int G = 32 / LPR;
    const int grp = lane / LPR, gl = lane % LPR;
    for (int i = grp; i - grp < rows; i += G) {   // every lane runs the same trips (rows is a multiple of G or smaller)
        const int64_t r = r0 + i;
        const bool live = i < rows && r < n_rows;
        int y = -1;
        if (live && gl == 0) {
            y = lab_s ? lab_s[i] : __ldg(p.labels + r);
            if (y >= p.cols) {
                latch(p.ctl, AA_ERR_BAD_INDEX);
                y = -1;
            }
        }
        RunState st = {-INFINITY, 0.0f};
        if (live) {
            const uint4* row = reinterpret_cast<const uint4*>(xs + (size_t)i * g.row_bytes);
#pragma unroll 2
            for (int v = gl; v < g.nvec; v += LPR) {
                float x[VE];
                Vec<T>::unpack(row[v], x);
                absorb_vec(st, x);
            }
        }
        st = group_merge<LPR>(st);
        if (live && gl == 0) {
            float loss = 0.0f;
            if (y >= 0) {
                const T* row_e = reinterpret_cast<const T*>(xs + (size_t)i * g.row_bytes);
                float x_y;
                if (sizeof(T) == 2) x_y = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(row_e)[y] << 16);
                else x_y = reinterpret_cast<const float*>(row_e)[y];
                loss = finish_row(st, x_y);
            }
            p.out[r] = loss;
        }
    }
}

template <typename T, int LPR>
__global__ void __launch_bounds__(kLossThreads, 1) row_loss_tma_kernel(LossParams p, LossGeometry g) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* ring = smem;
    LossRing* cb = reinterpret_cast<LossRing*>(smem + (size_t)g.stages * g.stage_bytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < g.stages; ++s) {
            mbar_init(&cb->full[s], 1);
            mbar_init(&cb->empty[s], kLSplit);
        }
        cb->stop_j = 0x7FFFFFFF;
        cb->abort_flag = 0;
        mbar_fence_init();
    }
    const int64_t n_rows = effective_rows(p);
    const long long n_units = (n_rows + g.chunk_rows - 1) / g.chunk_rows;
    volatile int* abort_flag = &cb->abort_flag;
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        const unsigned char* base = static_cast<const unsigned char*>(p.logits);
        const size_t stride_bytes = (size_t)p.row_stride * sizeof(T);
        const long long n_tickets = (n_units + kUnitsPerTicket - 1) / kUnitsPerTicket;
        int j = 0, stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        unsigned int next_ticket = 0;
        if (lane == 0) next_ticket = atomicAdd(&p.ctl->ticket, 1u);
        next_ticket = __shfl_sync(0xFFFFFFFFu, next_ticket, 0);
        while (ok && (long long)next_ticket < n_tickets) {
            const long long u0 = (long long)next_ticket * kUnitsPerTicket;
            if (lane == 0) next_ticket = atomicAdd(&p.ctl->ticket, 1u);   // lands while this ticket is issued
            for (int q = 0; q < kUnitsPerTicket; ++q) {
                const long long u = u0 + q;
                if (u >= n_units) break;
                if (j >= g.stages && !mbar_wait(&cb->empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                unsigned char* dst = ring + (size_t)stage * g.stage_bytes;
                {
                    const long long r0 = u * g.chunk_rows;
                    const int rows = (int)(n_rows - r0 < g.chunk_rows ? n_rows - r0 : g.chunk_rows);   // > 0
                    // the unit's labels ride along when the unit is full and their slice is 16-byte aligned
                    const uint32_t lab_bytes = (rows == g.chunk_rows && g.chunk_rows >= 4 && (((uintptr_t)(p.labels + r0)) & 15) == 0)
                                                   ? (uint32_t)g.chunk_rows * 4u : 0u;
                    if (lane == 0) {
                        cb->unit_of_stage[stage] = u;
                        cb->labels_staged[stage] = lab_bytes != 0;
                        mbar_arrive_expect_tx(&cb->full[stage], (uint32_t)rows * g.row_bytes + lab_bytes);
                        if (lab_bytes) bulk_g2s(&cb->labels[stage][0], p.labels + r0, lab_bytes, &cb->full[stage]);
                        if (g.contiguous) bulk_g2s(dst, base + (size_t)r0 * stride_bytes, (uint32_t)rows * g.row_bytes, &cb->full[stage]);
                    }
                    if (!g.contiguous) {
                        __syncwarp();
                        if (lane < rows) bulk_g2s(dst + (size_t)lane * g.row_bytes, base + (size_t)(r0 + lane) * stride_bytes, g.row_bytes, &cb->full[stage]);
                    }
                }
                __syncwarp();
                ++j;
                if (++stage == g.stages) { stage = 0; phase ^= 1u; }
            }
            next_ticket = __shfl_sync(0xFFFFFFFFu, next_ticket, 0);
        }
        if (ok) {
            // wake every consumer pair once with an empty stage
            if (lane == 0) *(volatile int*)&cb->stop_j = j;
            for (int c = 0; c < g.stages && ok; ++c) {
                if (j >= g.stages && !mbar_wait(&cb->empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                if (lane == 0) mbar_arrive(&cb->full[stage]);
                ++j;
                if (++stage == g.stages) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok) {
            if (lane == 0) loss_give_up(p, cb);
            const int pending = j < g.stages ? j : g.stages;
            for (int back = 1; back <= pending; ++back) {
                const int jj = j - back, st = jj % g.stages, use = jj / g.stages;
                const long long t0 = clock64();
                while (!mbar_try_wait(&cb->full[st], (uint32_t)(use & 1)) && clock64() - t0 < kWaitCycles) {}
            }
        }
    } else {
        // ------------------------------------------------------------ consumers
        const int cidx = warp - 1;
        const int stage = cidx / kLSplit, part = cidx - stage * kLSplit;
        if (stage < g.stages) {
            const unsigned char* xs = ring + (size_t)stage * g.stage_bytes;
            for (int n = 0;; ++n) {
                if (!mbar_wait(&cb->full[stage], (uint32_t)(n & 1), abort_flag)) {
                    if (lane == 0) loss_give_up(p, cb);
                    break;
                }
                const int j = n * g.stages + stage;
                if (j >= *(volatile int*)&cb->stop_j) break;
                const long long u = cb->unit_of_stage[stage];
                {
                    const int rows_per = g.chunk_rows / kLSplit;
                    const long long r0 = u * g.chunk_rows + part * rows_per;
                    const int* lab_s = cb->labels_staged[stage] ? &cb->labels[stage][part * rows_per] : nullptr;
                    consume_short<T, LPR>(p, g, xs + (size_t)part * rows_per * g.row_bytes, rows_per, r0, n_rows, lab_s, lane);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&cb->empty[stage]);
            }
        }
    }
    __syncthreads();
    if (tid == 0) {
        // last CTA out re-arms the ticket counter for the next kernel on this context
        __threadfence();
        const unsigned int prev = atomicAdd(&p.ctl->done, 1u);
        if (prev == gridDim.x - 1) {
            p.ctl->ticket = 0;
            p.ctl->done = 0;
        }
    }
}

int pow2_floor_l(int64_t v) {
    int q = 1;
    while ((int64_t)q * 2 <= v) q <<= 1;
    return q;
}

template <typename T>
const void* pick_loss_kernel(int lpr) {
    switch (lpr) {
        case 4: return (const void*)row_loss_tma_kernel<T, 4>;
        case 8: return (const void*)row_loss_tma_kernel<T, 8>;
        case 16: return (const void*)row_loss_tma_kernel<T, 16>;
        default: return (const void*)row_loss_tma_kernel<T, 32>;
    }
}

}  // namespace

aa_status launch_instance_loss_tma(aa_ctx_impl* c, const LossParams& p_in, int dtype) {
    LossParams p = p_in;
    const int es = dtype == AA_BF16 ? 2 : 4;
    const int64_t row_bytes = p.cols * es;
    if ((uintptr_t)p.logits % 16 || (p.row_stride * es) % 16 || row_bytes % 16 || row_bytes < 256) return AA_ERR_UNSUPPORTED;
    if ((uintptr_t)p.labels % 4) return AA_ERR_UNSUPPORTED;
    LossGeometry g = {};
    g.row_bytes = (uint32_t)row_bytes;
    g.nvec = (int)(row_bytes / 16);
    if (row_bytes * 2 > kLTargetStage + 8 * 1024) return AA_ERR_UNSUPPORTED;      // a stage holds at least two rows
    if (p.rows * row_bytes < kMinRingBytes) return AA_ERR_UNSUPPORTED;
    // rows of up to 4 KB: the load-based kernel (a warp or less per row, four vectors per trip) is ahead since its
    // running-maximum bookkeeping was shared between vectors (1000 fp32 classes: 5.8 against 5.1 TB/s; 1 KB rows: 4.6 against 2.8)
    if (row_bytes <= 4096) return AA_ERR_UNSUPPORTED;
    g.chunk_rows = pow2_floor_l((kLTargetStage + 8 * 1024) / row_bytes);
    if (g.chunk_rows > 32) g.chunk_rows = 32;
    g.stage_bytes = (int)(((int64_t)g.chunk_rows * row_bytes + 127) / 128 * 128);
    g.contiguous = p.row_stride == p.cols ? 1 : 0;
    const int rows_per = g.chunk_rows / kLSplit;
    int lpr = 4;
    while (lpr < 32 && lpr * 2 <= g.nvec) lpr <<= 1;          // at least two vectors per lane
    if (32 / lpr > rows_per) lpr = 32 / rows_per;
    const size_t fixed = sizeof(LossRing) + 128;
    const size_t budget = 220 * 1024;
    int stages = (int)((budget - fixed) / g.stage_bytes);
    if (stages > kLMaxStages) stages = kLMaxStages;
    if (stages < 2) return AA_ERR_UNSUPPORTED;
    g.stages = stages;
    const size_t smem = fixed + (size_t)stages * g.stage_bytes;

    const int64_t n_units = (p.rows + g.chunk_rows - 1) / g.chunk_rows;
    const int64_t n_tickets = (n_units + kUnitsPerTicket - 1) / kUnitsPerTicket;
    if (n_tickets > 0x7FFFFFFFll) return AA_ERR_UNSUPPORTED;
    int grid = c->sm_count;
    if (grid > n_tickets) grid = (int)n_tickets;
    if (grid < 1) grid = 1;
    const void* kernel = dtype == AA_BF16 ? pick_loss_kernel<uint16_t>(lpr) : pick_loss_kernel<float>(lpr);
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return AA_ERR_CUDA;
    void* args[] = {&p, &g};
    if (cudaLaunchKernel(kernel, dim3(grid), dim3(kLossThreads), args, smem, c->stream) != cudaSuccess) return AA_ERR_CUDA;
    ++c->launches;
    return AA_OK;
}

}  // namespace aa
