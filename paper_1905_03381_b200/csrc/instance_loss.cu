// Per-instance Boss loss from logits (Sec. "Asynchronous joint learning with CPU/GPU": the loss f pushed with each index i).
//
// Row cross-entropy  l_r = log sum_c exp(x_rc) - x_{r,y_r}  in a single pass over the row:
// every thread keeps a running maximum M and a sum S of 2^(t - M) over its elements, with
// t = x * log2(e), so that sum_c 2^(t_c) = S * 2^M; thread states are merged by warp shuffles
// (and through shared memory when a CTA shares a row).  For sequence tasks the token rows of
// a sentence are then summed in row order (fp64 accumulator) by a second small kernel.
#include "loss_common.cuh"

namespace aa {

namespace {

constexpr int kRowThreads = 256;   // CTA size when one CTA owns a row and rows are few
constexpr int kRowThreadsMany = 128;   // ... and when there are many rows per resident CTA

// Accumulate the elements [j0, j1) of one row, strided over `nthreads` workers starting at `rank`.
// Handles any alignment: scalar head up to the first 16-byte boundary, vector body, scalar tail.
template <typename T>
__device__ __forceinline__ void scan_row(RunState& st, const T* row, int64_t cols, int rank, int nthreads) {
    constexpr int VE = Vec<T>::kElems;
    const uintptr_t addr = (uintptr_t)row;
    int64_t head = ((16 - (addr & 15)) & 15) / sizeof(T);
    if (head > cols) head = cols;
    const int64_t nvec = (cols - head) / VE;
    const int64_t tail0 = head + nvec * VE;
    const T* body = row + head;
    constexpr int K = 4;                    // vectors per trip that share the running-maximum bookkeeping
    int64_t v = rank;
    for (; v + (K - 1) * (int64_t)nthreads < nvec; v += K * (int64_t)nthreads) {
        float x[K][VE];
#pragma unroll
        for (int k = 0; k < K; ++k) Vec<T>::load(body + (v + k * (int64_t)nthreads) * VE, x[k]);
        absorb_vecs<K, VE>(st, x);
    }
    for (; v + (int64_t)nthreads < nvec; v += 2 * (int64_t)nthreads) {
        float x[2][VE];
        Vec<T>::load(body + v * VE, x[0]);
        Vec<T>::load(body + (v + nthreads) * VE, x[1]);
        absorb_vecs<2, VE>(st, x);
    }
    for (; v < nvec; v += nthreads) {
        float x[VE];
        Vec<T>::load(body + v * VE, x);
        absorb_vec(st, x);
    }
    // the few unaligned elements at both ends
    for (int64_t j = rank; j < head; j += nthreads) {
        const float t = Vec<T>::one(row + j) * kLog2e;
        absorb(st, &t, 1);
    }
    for (int64_t j = tail0 + rank; j < cols; j += nthreads) {
        const float t = Vec<T>::one(row + j) * kLog2e;
        absorb(st, &t, 1);
    }
}

// Short rows: LPR lanes per row, several rows per warp.
template <typename T, int LPR>
__global__ void __launch_bounds__(256, sizeof(T) == 4 ? 6 : 4) row_loss_group_kernel(LossParams p) {
    grid_dependency_wait();      // the row count and the logits may come from the previous kernel of the stream
    grid_dependency_release();
    const int64_t rows = effective_rows(p);
    const int gl = threadIdx.x % LPR;
    const int64_t groups_per_grid = (int64_t)gridDim.x * (blockDim.x / LPR);
    const int64_t group0 = (int64_t)blockIdx.x * (blockDim.x / LPR) + threadIdx.x / LPR;
    // whole warps iterate together so that the shuffles see every lane
    const int64_t rounds = (rows + groups_per_grid - 1) / groups_per_grid;
    for (int64_t it = 0; it < rounds; ++it) {
        const int64_t r = group0 + it * groups_per_grid;
        RunState st = {-INFINITY, 0.0f};
        int y = -1;
        int64_t src = -1;
        if (r < rows) {
            src = source_row(p, r);
            if (src >= 0) y = checked_label(p, src);
            if (y >= 0) scan_row<T>(st, static_cast<const T*>(p.logits) + src * p.row_stride, p.cols, gl, LPR);
        }
        st = group_merge<LPR>(st);
        if (gl == 0 && r < rows) {
            float loss = 0.0f;
            if (y >= 0) loss = finish_row(st, Vec<T>::one(static_cast<const T*>(p.logits) + src * p.row_stride + y));
            p.out[r] = loss;
        }
    }
}

// Very short aligned rows (at most kShortVecs 16-byte vectors per lane): the whole row sits in registers, so the row
// maximum is taken first and the sum second (no running rescale), and the loads of a row - label, every vector, and the
// device row count - are all issued before anything is consumed: one memory round trip, then the label's logit from L1.
constexpr int kShortVecs = 4;
template <typename T, int LPR>
__global__ void __launch_bounds__(256) row_loss_short_kernel(LossParams p) {
    constexpr int VE = Vec<T>::kElems;
    grid_dependency_wait();      // the row count and the logits may come from the previous kernel of the stream
    grid_dependency_release();
    const int64_t rows_host = p.rows;
    int64_t rows = rows_host;
    int32_t count_raw = 0;
    if (p.count_dev) count_raw = __ldg(p.count_dev);
    const int gl = threadIdx.x % LPR;
    const int nvec = (int)(p.cols / VE);
    const int64_t groups_per_grid = (int64_t)gridDim.x * (blockDim.x / LPR);
    const int64_t group0 = (int64_t)blockIdx.x * (blockDim.x / LPR) + threadIdx.x / LPR;
    const int64_t rounds = (rows_host + groups_per_grid - 1) / groups_per_grid;
    const T* base = static_cast<const T*>(p.logits);
    for (int64_t it = 0; it < rounds; ++it) {
        const int64_t r = group0 + it * groups_per_grid;
        const bool inb = r < rows_host;
        const T* row = base + (inb ? r : 0) * p.row_stride;
        int y = inb ? __ldg(p.labels + r) : -1;
        float x[kShortVecs][VE];
#pragma unroll
        for (int q = 0; q < kShortVecs; ++q) {
            const int v = gl + q * LPR;
            if (inb && v < nvec) {
                Vec<T>::load(row + (int64_t)v * VE, x[q]);
            } else {
#pragma unroll
                for (int e = 0; e < VE; ++e) x[q][e] = -INFINITY;
            }
        }
        if (p.count_dev) rows = count_raw < 0 ? 0 : ((int64_t)count_raw < rows_host ? (int64_t)count_raw : rows_host);
        const bool live = r < rows;
        if (live && y >= p.cols) {
            latch(p.ctl, AA_ERR_BAD_INDEX);
            y = -1;
        }
        const float label_logit = (live && y >= 0) ? Vec<T>::one(row + y) : 0.0f;
        float m = -INFINITY;
#pragma unroll
        for (int q = 0; q < kShortVecs; ++q)
#pragma unroll
            for (int e = 0; e < VE; ++e) m = fmaxf(m, x[q][e]);
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
        const float neg_ref = m == -INFINITY ? 0.0f : -m * kLog2e;
        float s0 = 0.0f, s1 = 0.0f;
#pragma unroll
        for (int q = 0; q < kShortVecs; ++q)
#pragma unroll
            for (int e = 0; e < VE; e += 2) {
                s0 += ex2_approx(fmaf(x[q][e], kLog2e, neg_ref));
                s1 += ex2_approx(fmaf(x[q][e + 1], kLog2e, neg_ref));
            }
        float ssum = s0 + s1;
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) ssum += __shfl_xor_sync(0xFFFFFFFFu, ssum, o);
        if (gl == 0 && live) {
            RunState st = {m * kLog2e, ssum};
            p.out[r] = y >= 0 ? finish_row(st, label_logit) : 0.0f;
        }
    }
}

// Long rows: one CTA per row.  1536 threads per SM (40 registers: the four-vector trips would take 48 and leave 1280):
// twelve CTAs of 128 threads when there are rows enough to keep them all busy (the merge at the end of a row then
// idles a smaller part of the SM: 25,000 x 32,000 bf16 runs at 6.1 instead of 5.7 TB/s), six of 256 otherwise.
template <typename T, int THREADS>
__global__ void __launch_bounds__(THREADS, 1536 / THREADS) row_loss_cta_kernel(LossParams p) {
    constexpr int kRowThreads = THREADS;
    __shared__ RunState warp_state[kRowThreads / 32];
    __shared__ unsigned int s_row[2];
    grid_dependency_wait();      // the row count and the logits may come from the previous kernel of the stream
    grid_dependency_release();
    const int64_t rows = effective_rows(p);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Rows are handed out by the ticket counter (the first row of a CTA is its block index, the request for the row
    // after next is in flight while a row is scanned), so that CTAs finish within one row of each other.
    if (threadIdx.x == 0) {
        s_row[0] = blockIdx.x;
        s_row[1] = gridDim.x + atomicAdd(&p.ctl->ticket, 1u);
    }
    __syncthreads();
    for (int it = 0;; ++it) {
        const int64_t r = s_row[it & 1];
        if (r >= rows) break;
        unsigned int fresh = 0;
        if (threadIdx.x == 0) fresh = gridDim.x + atomicAdd(&p.ctl->ticket, 1u);
        const int64_t src = source_row(p, r);                 // uniform over the CTA
        const int y = src >= 0 ? checked_label(p, src) : -1;
        const T* row = static_cast<const T*>(p.logits) + (src >= 0 ? src : 0) * p.row_stride;
        RunState st = {-INFINITY, 0.0f};
        if (y >= 0) scan_row<T>(st, row, p.cols, threadIdx.x, kRowThreads);
        st = group_merge<32>(st);
        if (lane == 0) warp_state[warp] = st;
        __syncthreads();                       // every thread has read this iteration's slot of s_row
        if (threadIdx.x == 0) s_row[it & 1] = fresh;
        if (warp == 0) {
            RunState t = lane < kRowThreads / 32 ? warp_state[lane] : RunState{-INFINITY, 0.0f};
            t = group_merge<32>(t);
            if (lane == 0) p.out[r] = y >= 0 ? finish_row(t, Vec<T>::one(row + y)) : 0.0f;
        }
        __syncthreads();
    }
    // last CTA out re-arms the ticket counter for the next kernel on this context
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int prev = atomicAdd(&p.ctl->done, 1u);
        if (prev == gridDim.x - 1) {
            p.ctl->ticket = 0;
            p.ctl->done = 0;
        }
    }
}

// Per-sentence sums of token-row losses, one warp per segment, rows added in fp64.
__global__ void __launch_bounds__(256) segment_sum_kernel(const float* __restrict__ row_loss, const int32_t* __restrict__ offsets,
                                                          int64_t n_seg, int64_t rows, float* __restrict__ out, Control* ctl) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t s = warp; s < n_seg; s += nwarps) {
        const int64_t a = __ldg(offsets + s), b = __ldg(offsets + s + 1);
        double acc = 0.0;
        if (a < 0 || b < a || b > rows) {
            if (lane == 0) latch(ctl, AA_ERR_BAD_INDEX);
        } else {
            for (int64_t r = a + lane; r < b; r += 32) acc += (double)row_loss[r];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) out[s] = (float)acc;
    }
}

template <typename T>
aa_status launch_rows(aa_ctx_impl* c, LossParams& p) {
    const int es = (int)sizeof(T);
    const int64_t row_bytes = p.cols * es;
    void* args[] = {&p};
    const void* kernel;
    int threads, grid;
    // Up to 32 KB a warp (or part of one) owns a row: no CTA barrier per row, and with four vectors per trip that beats
    // both a CTA per row and a bulk-copy ring with consumer warps (which this library had for 4-16 KB rows: 5.1-5.5 TB/s
    // against 5.6-6.8 here).  Longer rows take a CTA each.
    if (row_bytes > 32 * 1024) {
        const bool many = p.rows >= 4ll * (1536 / kRowThreadsMany) * c->sm_count;
        kernel = many ? (const void*)row_loss_cta_kernel<T, kRowThreadsMany> : (const void*)row_loss_cta_kernel<T, kRowThreads>;
        threads = many ? kRowThreadsMany : kRowThreads;
        int cap = resident_ctas(c, kernel, threads, 0);
        if (cap <= 0) return AA_ERR_CUDA;
        grid = (int)(p.rows < cap ? p.rows : cap);
    } else {
        const int64_t work = (row_bytes + 15) / 16;   // 16-byte vectors per row
        int lpr = 2;
        while (lpr < 32 && lpr * 4 <= work) lpr <<= 1;   // two to four vectors per lane
        threads = 256;
        const bool short_rows = !p.row_idx && row_bytes % 16 == 0 && (uintptr_t)p.logits % 16 == 0 && (p.row_stride * es) % 16 == 0 &&
                                work <= (int64_t)lpr * kShortVecs;
        if (short_rows) {
            switch (lpr) {
                case 2: kernel = (const void*)row_loss_short_kernel<T, 2>; break;
                case 4: kernel = (const void*)row_loss_short_kernel<T, 4>; break;
                case 8: kernel = (const void*)row_loss_short_kernel<T, 8>; break;
                case 16: kernel = (const void*)row_loss_short_kernel<T, 16>; break;
                default: kernel = (const void*)row_loss_short_kernel<T, 32>; lpr = 32; break;
            }
        } else
        switch (lpr) {
            case 2: kernel = (const void*)row_loss_group_kernel<T, 2>; break;
            case 4: kernel = (const void*)row_loss_group_kernel<T, 4>; break;
            case 8: kernel = (const void*)row_loss_group_kernel<T, 8>; break;
            case 16: kernel = (const void*)row_loss_group_kernel<T, 16>; break;
            default: kernel = (const void*)row_loss_group_kernel<T, 32>; lpr = 32; break;
        }
        int cap = resident_ctas(c, kernel, threads, 0);
        if (cap <= 0) return AA_ERR_CUDA;
        const int64_t rows_per_cta = threads / lpr;
        const int64_t want = (p.rows + rows_per_cta - 1) / rows_per_cta;
        grid = (int)(want < cap ? want : cap);
    }
    if (grid < 1) grid = 1;
    if (launch_overlapped(c, kernel, dim3(grid), dim3(threads), args, 0, false) != cudaSuccess) return AA_ERR_CUDA;
    ++c->launches;
    return AA_OK;
}

}  // namespace

aa_status launch_instance_loss(aa_ctx_impl* c, const aa_logits& lg, const int32_t* labels, const int32_t* offsets,
                               int64_t n_seg, const int32_t* count_dev, float* out_loss, const int32_t* row_idx, int64_t n_rows) {
    LossParams p;
    p.logits = lg.data;
    p.rows = row_idx ? n_rows : lg.rows;
    p.row_idx = row_idx;
    p.n_stored = lg.rows;
    p.cols = lg.cols;
    p.row_stride = lg.row_stride;
    p.labels = labels;
    p.count_dev = offsets ? nullptr : count_dev;
    p.ctl = c->ctl;
    p.out = offsets ? c->row_scratch : out_loss;
    if (p.rows > 0) {
        const aa_status st = lg.dtype == AA_BF16 ? launch_rows<uint16_t>(c, p) : launch_rows<float>(c, p);
        if (st != AA_OK) return st;
    }
    if (offsets && n_seg > 0) {
        const float* row_loss = c->row_scratch;
        int64_t rows = p.rows;
        Control* ctl = c->ctl;
        void* args[] = {&row_loss, &offsets, &n_seg, &rows, &out_loss, &ctl};
        const int64_t want = (n_seg + 7) / 8;   // 8 warps per CTA
        const int cap = c->sm_count * 8;
        const int grid = (int)(want < cap ? want : cap);
        if (cudaLaunchKernel((const void*)segment_sum_kernel, dim3(grid), dim3(256), args, 0, c->stream) != cudaSuccess)
            return AA_ERR_CUDA;
        ++c->launches;
    }
    return AA_OK;
}

}  // namespace aa
