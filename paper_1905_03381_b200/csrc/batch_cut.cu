// Batch cut + cursor: turns the ordered survivor list of a screened pool into the batch that
// Algorithm 1 (Assistant.sample_batch) would have returned, and tells how far it walked.
//
// Algorithm 1 appends accepted instances until the batch holds batch_size of them, so its batch is
// the first batch_size survivors of the list and its walk ends right after the last one taken.
// For sequence tasks the batch is bounded by a token budget instead (Sec. "Machine Translation" trains on batches of
// a given number of tokens): the longest prefix of survivors whose lengths add up to at most the
// budget, together with the running token offsets that the per-sentence loss needs.
// One CTA: the lengths of up to a million survivors are scanned in chunks of 1024 with a carry.
#include "aa_internal.cuh"

namespace aa {

namespace {

constexpr int kCutThreads = 1024;

struct CutParams {
    const int32_t* idx;
    const int32_t* count_dev;
    int64_t m_host;          // entries idx can hold (bound on the device count)
    int64_t n_cand;          // candidates in the screened pool
    int64_t n_stored;        // rows `lengths` covers
    int64_t batch_size;      // 0 = no limit on instances
    const int32_t* lengths;  // nullable
    int64_t token_budget;    // used when lengths != nullptr
    int32_t* out_m;
    int32_t* out_consumed;
    int32_t* out_offsets;    // nullable, offsets_capacity entries
    int64_t offsets_capacity;
    Control* ctl;
};

__global__ void __launch_bounds__(kCutThreads) batch_cut_kernel(CutParams p) {
    __shared__ long long warp_sum[kCutThreads / 32];
    __shared__ long long carry_s;
    __shared__ int taken_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int64_t m = p.m_host;
    if (p.count_dev) {
        const int64_t c = *p.count_dev;
        m = c < 0 ? 0 : (c < m ? c : m);
    }
    int64_t cap = m;                                            // survivors that may enter the batch
    if (p.batch_size > 0 && p.batch_size < cap) cap = p.batch_size;
    int64_t b = cap;
    if (p.lengths) {
        if (tid == 0) { carry_s = 0; taken_s = 0; }
        if (tid == 0 && p.out_offsets && p.offsets_capacity > 0) p.out_offsets[0] = 0;
        __syncthreads();
        bool full = false;                                      // the budget is used up: later survivors cannot enter
        for (int64_t k0 = 0; k0 < cap && !full; k0 += kCutThreads) {
            const int64_t k = k0 + tid;
            long long len = 0;
            if (k < cap) {
                const long long r = p.idx[k];
                if ((unsigned long long)r < (unsigned long long)p.n_stored) {
                    const int v = p.lengths[r];
                    len = v > 0 ? v : 0;
                } else {
                    latch(p.ctl, AA_ERR_BAD_INDEX);
                }
            }
            // inclusive scan of the chunk
            long long inc = len;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const long long t = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                if (lane >= o) inc += t;
            }
            if (lane == 31) warp_sum[warp] = inc;
            __syncthreads();
            long long before = carry_s;
            for (int w = 0; w < warp; ++w) before += warp_sum[w];
            const long long cum = before + inc;                 // tokens of survivors 0..k
            const bool fits = k < cap && cum <= p.token_budget;
            if (fits && p.out_offsets && k + 1 < p.offsets_capacity) p.out_offsets[k + 1] = (int32_t)cum;
            const int n_fit = __syncthreads_count(fits);        // lengths are non-negative: the fitting survivors are a prefix
            if (tid == 0) {
                taken_s += n_fit;
                long long total = carry_s;
                for (int w = 0; w < kCutThreads / 32; ++w) total += warp_sum[w];
                carry_s = total;
            }
            full = n_fit < kCutThreads && k0 + n_fit < cap;
            __syncthreads();
        }
        b = taken_s;
    }
    if (tid == 0) {
        *p.out_m = (int32_t)b;
        // the walk ends right after the last instance taken; if the survivors ran out first it covered the whole pool
        const bool limited = b < m || (p.batch_size > 0 && b == p.batch_size);
        long long consumed = p.n_cand;
        if (limited) consumed = b > 0 ? (long long)p.idx[b - 1] + 1 : 0;
        *p.out_consumed = (int32_t)consumed;
    }
}

}  // namespace

aa_status launch_batch_cut(aa_ctx_impl* c, const int32_t* idx, const int32_t* count_dev, int64_t m_host, int64_t n_cand,
                           int64_t n_stored, int64_t batch_size, const int32_t* lengths, int64_t token_budget, int32_t* out_m,
                           int32_t* out_consumed, int32_t* out_offsets, int64_t offsets_capacity) {
    CutParams p = {idx, count_dev, m_host, n_cand, n_stored, batch_size, lengths, token_budget,
                   out_m, out_consumed, out_offsets, offsets_capacity, c->ctl};
    void* args[] = {&p};
    if (cudaLaunchKernel((const void*)batch_cut_kernel, dim3(1), dim3(kCutThreads), args, 0, c->stream) != cudaSuccess) return AA_ERR_CUDA;
    ++c->launches;
    return AA_OK;
}

}  // namespace aa
