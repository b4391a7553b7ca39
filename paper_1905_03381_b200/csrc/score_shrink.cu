// Assistant score -> Bernoulli shrink -> ordered batch list, fused in one pass
// (Algorithm 1, Assistant.sample_batch, evaluated for a whole candidate pool at once).
//
// The kernels in this file read the features with ordinary 128-bit (or element-wise) loads:
// any alignment, any stride, CSR rows, or precomputed pre-activations.  A CTA repeatedly takes
// the next tile of candidates from the ticket counter, computes the tile's pre-activations
// into shared memory, then draws the keep/skip decisions and appends the kept candidates
// (scan_tail.cuh).  Aligned dense rows normally take the bulk-copy kernel of
// score_shrink_tma.cu instead.
#include <string.h>

#include <mutex>

#include "scan_tail.cuh"

namespace aa {

namespace {

struct TailSmem {
    float s[kMaxTileRows];     // pre-activation per candidate of the tile
    unsigned int mask[32];     // keep ballot per 32-candidate unit
    int off[32];               // exclusive prefix of the unit counts inside the tile
    int base;                  // kept candidates in all earlier tiles
    unsigned int tile;
};

// Shrink decision + ordered append for one tile whose pre-activations are in sm.s.
// All threads of the CTA call this; contains CTA barriers.
__device__ void shrink_compact_tile(const ShrinkParams& p, unsigned int tile, unsigned int epoch, TailSmem& sm) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const int units = p.tile_rows >> 5;
    const long long k0 = (long long)tile * p.tile_rows;

    for (int u = warp; u < units; u += nwarps) {
        const long long k = k0 + u * 32 + lane;
        bool keep = false;
        if (k < p.n_cand) {
            const float s = sm.s[u * 32 + lane];
            keep = keep_decision(p, k, s);
            if (p.out_score) p.out_score[k] = s;
            if (p.out_mask) p.out_mask[k] = keep ? 1 : 0;
        }
        const unsigned int m = __ballot_sync(0xFFFFFFFFu, keep);
        if (lane == 0) sm.mask[u] = m;
    }
    __syncthreads();
    if (warp == 0) {
        const int cnt = lane < units ? __popc(sm.mask[lane]) : 0;
        int inc = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, inc, o);
            if (lane >= o) inc += t;
        }
        sm.off[lane] = inc - cnt;
        const int total = __shfl_sync(0xFFFFFFFFu, inc, 31);
        const int base = lookback_exclusive(p, tile, epoch, total);
        if (lane == 0) {
            sm.base = base;
            if (tile == p.n_tiles - 1) *p.out_count = base + total;
        }
    }
    __syncthreads();
    for (int u = warp; u < units; u += nwarps) {
        const unsigned int m = sm.mask[u];
        if ((m >> lane) & 1u) {
            const long long k = k0 + u * 32 + lane;
            const long long pos = (long long)sm.base + sm.off[u] + __popc(m & ((1u << lane) - 1u));
            if (pos < p.capacity) p.out_idx[pos] = p.row_idx ? p.row_idx[k] : (int32_t)k;
            else latch(p.ctl, AA_ERR_CAPACITY);
        }
    }
}

__device__ __forceinline__ bool next_tile(const ShrinkParams& p, TailSmem& sm, unsigned int& tile) {
    __syncthreads();   // previous tile's readers of sm are done
    if (threadIdx.x == 0) sm.tile = atomicAdd(&p.ctl->ticket, 1u);
    __syncthreads();
    tile = sm.tile;
    return tile < p.n_tiles;
}

constexpr float kNaN = __builtin_nanf("");

// ---------------------------------------------------------------- dense linear Assistant
// LPR lanes cooperate on one row.  VEC: rows are 16-byte aligned, d is a whole number of
// vectors and w sits in shared memory in the conflict-free vector layout.
template <typename T, int LPR, bool VEC>
__global__ void __launch_bounds__(kScanThreads) score_shrink_dense_kernel(DenseFeat f, ShrinkParams p, int w_in_smem) {
    extern __shared__ __align__(16) float w_smem[];
    __shared__ TailSmem sm;
    constexpr int VE = Vec<T>::kElems;
    const int tid = threadIdx.x;
    const int nvec = (int)(f.d / VE);
    const float* wv = f.w;
    if (w_in_smem) {
        if (VEC) for (int j = tid; j < f.d; j += kScanThreads) w_smem[Vec<T>::w_index(j, nvec)] = f.w[j];
        else for (int j = tid; j < f.d; j += kScanThreads) w_smem[j] = f.w[j];
        wv = w_smem;
    }
    const float bias = *f.b;
    const unsigned int epoch = read_epoch(p);
    const T* base = static_cast<const T*>(f.base);
    constexpr int G = kScanThreads / LPR;
    const int group = tid / LPR, gl = tid % LPR;

    unsigned int tile;
    while (next_tile(p, sm, tile)) {
        const long long k0 = (long long)tile * p.tile_rows;
        for (int rl = group; rl < p.tile_rows; rl += G) {
            const long long k = k0 + rl;
            const long long r = k < p.n_cand ? candidate_row(p, k) : -1;
            float acc = 0.0f;
            if (r >= 0) {
                const T* row = base + r * f.row_stride;
                if (VEC) {
#pragma unroll 4
                    for (int v = gl; v < nvec; v += LPR) {
                        float x[VE], wq[VE];
                        Vec<T>::load(row + (long long)v * VE, x);
                        Vec<T>::load_w(w_smem, nvec, v, wq);
#pragma unroll
                        for (int e = 0; e < VE; ++e) acc = fmaf(x[e], wq[e], acc);
                    }
                } else {
                    for (long long j = gl; j < f.d; j += LPR) acc = fmaf(Vec<T>::one(row + j), wv[j], acc);
                }
            }
#pragma unroll
            for (int o = LPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
            if (gl == 0) sm.s[rl] = r >= 0 ? acc + bias : kNaN;
        }
        __syncthreads();
        shrink_compact_tile(p, tile, epoch, sm);
    }
    scan_epilogue(p, epoch);
}

// ---------------------------------------------------------------- CSR bag-of-words Assistant
constexpr int kCsrUnroll = 8;
template <int LPR>
__global__ void __launch_bounds__(kScanThreads) score_shrink_csr_kernel(CsrFeat f, ShrinkParams p) {
    __shared__ TailSmem sm;
    const int tid = threadIdx.x;
    const float bias = *f.b;
    const unsigned int epoch = read_epoch(p);
    constexpr int G = kScanThreads / LPR;
    const int group = tid / LPR, gl = tid % LPR;

    unsigned int tile;
    while (next_tile(p, sm, tile)) {
        const long long k0 = (long long)tile * p.tile_rows;
        for (int rl = group; rl < p.tile_rows; rl += G) {
            const long long k = k0 + rl;
            const long long r = k < p.n_cand ? candidate_row(p, k) : -1;
            float acc = 0.0f;
            if (r >= 0) {
                const int e0 = __ldg(f.indptr + r), e1 = __ldg(f.indptr + r + 1);
                // kCsrUnroll entries per lane and trip: their column/value loads, then their weight gathers, are in
                // flight together (the row is a chain of three dependent memory round trips, not one per entry)
                for (int e = e0 + gl; e < e1; e += kCsrUnroll * LPR) {
                    int c[kCsrUnroll];
                    float v[kCsrUnroll];
#pragma unroll
                    for (int u = 0; u < kCsrUnroll; ++u) {
                        const int ee = e + u * LPR;
                        const bool in = ee < e1;
                        c[u] = in ? __ldg(f.col + ee) : 0;
                        v[u] = in ? __ldg(f.val + ee) : 0.0f;
                    }
                    float wq[kCsrUnroll];
                    bool bad = false;
#pragma unroll
                    for (int u = 0; u < kCsrUnroll; ++u) {
                        const bool ok = (unsigned long long)(unsigned int)c[u] < (unsigned long long)f.d;
                        bad |= !ok;
                        wq[u] = ok ? __ldg(f.w + c[u]) : 0.0f;
                    }
#pragma unroll
                    for (int u = 0; u < kCsrUnroll; ++u) acc = fmaf(v[u], wq[u], acc);
                    if (bad) latch(p.ctl, AA_ERR_BAD_INDEX);
                }
            }
#pragma unroll
            for (int o = LPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
            if (gl == 0) sm.s[rl] = r >= 0 ? acc + bias : kNaN;
        }
        __syncthreads();
        shrink_compact_tile(p, tile, epoch, sm);
    }
    scan_epilogue(p, epoch);
}

// ---------------------------------------------------------------- precomputed pre-activations
__global__ void __launch_bounds__(kScanThreads) shrink_from_scores_kernel(const float* __restrict__ score, ShrinkParams p) {
    __shared__ TailSmem sm;
    const unsigned int epoch = read_epoch(p);
    unsigned int tile;
    while (next_tile(p, sm, tile)) {
        const long long k0 = (long long)tile * p.tile_rows;
        for (int rl = threadIdx.x; rl < p.tile_rows; rl += kScanThreads) {
            const long long k = k0 + rl;
            sm.s[rl] = k < p.n_cand ? __ldg(score + k) : 0.0f;
        }
        __syncthreads();
        shrink_compact_tile(p, tile, epoch, sm);
    }
    scan_epilogue(p, epoch);
}

int pow2_ceil(int64_t v) {
    int p = 1;
    while (p < v) p <<= 1;
    return p;
}

// Rows per tile: about `target_bytes` of input per tile, a multiple of 32, and small enough
// that the pool splits into at least two tiles per SM when it is large enough to.
int choose_tile_rows(const aa_ctx_impl* c, int64_t n_cand, double bytes_per_row, double target_bytes) {
    int64_t rows = (int64_t)(target_bytes / (bytes_per_row > 1.0 ? bytes_per_row : 1.0));
    const int64_t spread = n_cand / (2 * (int64_t)c->sm_count);
    if (rows > spread) rows = spread;
    rows = (rows / 32) * 32;
    if (rows < 32) rows = 32;
    if (rows > kMaxTileRows) rows = kMaxTileRows;
    return (int)rows;
}

template <typename K>
aa_status launch_scan(aa_ctx_impl* c, K kernel, size_t smem, const ShrinkParams& sp, void** args) {
    if (smem > 48 * 1024) {
        if (cudaFuncSetAttribute((const void*)kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return AA_ERR_CUDA;
    }
    int grid = resident_ctas(c, (const void*)kernel, kScanThreads, smem);
    if (grid <= 0) return AA_ERR_CUDA;
    if ((unsigned int)grid > sp.n_tiles) grid = (int)sp.n_tiles;
    if (cudaLaunchKernel((const void*)kernel, dim3(grid), dim3(kScanThreads), args, smem, c->stream) != cudaSuccess)
        return AA_ERR_CUDA;
    ++c->launches;
    return AA_OK;
}

template <typename T, bool VEC>
aa_status dispatch_dense(aa_ctx_impl* c, DenseFeat& f, ShrinkParams& sp, int lpr, size_t smem, int w_in_smem) {
    void* args[] = {&f, &sp, &w_in_smem};
    switch (lpr) {
        case 4: return launch_scan(c, score_shrink_dense_kernel<T, 4, VEC>, smem, sp, args);
        case 8: return launch_scan(c, score_shrink_dense_kernel<T, 8, VEC>, smem, sp, args);
        case 16: return launch_scan(c, score_shrink_dense_kernel<T, 16, VEC>, smem, sp, args);
        default: return launch_scan(c, score_shrink_dense_kernel<T, 32, VEC>, smem, sp, args);
    }
}

}  // namespace

aa_status finish_shrink_params(aa_ctx_impl* c, ShrinkParams& sp, int tile_rows) {
    sp.tile_rows = tile_rows;
    const int64_t n_tiles = (sp.n_cand + tile_rows - 1) / tile_rows;
    if (n_tiles > c->max_tiles) return AA_ERR_WORKSPACE;
    sp.n_tiles = (unsigned int)n_tiles;
    sp.ctl = c->ctl;
    sp.tile_state = c->tile_state;
    // flag generations repeat after 2^30 scans: clear the flags long before that can matter
    if (++c->scans_since_clear >= (1ull << 29)) {
        c->scans_since_clear = 0;
        if (cudaMemsetAsync(c->tile_state, 0, sizeof(unsigned long long) * c->max_tiles, c->stream) != cudaSuccess)
            return AA_ERR_CUDA;
    }
    return AA_OK;
}

aa_status launch_score_shrink_dense(aa_ctx_impl* c, const DenseFeat& f_in, ShrinkParams sp) {
    DenseFeat f = f_in;
    const int es = f.dtype == AA_BF16 ? 2 : 4;
    const int ve = 16 / es;
    const bool aligned = ((uintptr_t)f.base % 16 == 0) && ((f.row_stride * es) % 16 == 0) && (f.d % ve == 0);
    if (aligned) {
        aa_status st = launch_score_shrink_dense_tma(c, f, sp);
        if (st != AA_ERR_UNSUPPORTED) return st;
    }
    // the vector path keeps w in shared memory; otherwise rows are read element by element
    const bool vec = aligned && f.d * sizeof(float) <= 96 * 1024;
    const int64_t work_items = vec ? f.d / ve : f.d;
    int lpr = pow2_ceil((work_items + 1) / 2);
    lpr = lpr < 4 ? 4 : (lpr > 32 ? 32 : lpr);
    aa_status st = finish_shrink_params(c, sp, choose_tile_rows(c, sp.n_cand, (double)f.d * es, 192.0 * 1024));
    if (st != AA_OK) return st;
    const int w_in_smem = f.d * sizeof(float) <= 96 * 1024 ? 1 : 0;
    const size_t smem = w_in_smem ? (size_t)f.d * sizeof(float) : 0;
    if (f.dtype == AA_BF16)
        return vec ? dispatch_dense<uint16_t, true>(c, f, sp, lpr, smem, w_in_smem)
                   : dispatch_dense<uint16_t, false>(c, f, sp, lpr, smem, w_in_smem);
    return vec ? dispatch_dense<float, true>(c, f, sp, lpr, smem, w_in_smem)
               : dispatch_dense<float, false>(c, f, sp, lpr, smem, w_in_smem);
}

aa_status launch_score_shrink_csr(aa_ctx_impl* c, const CsrFeat& f_in, ShrinkParams sp) {
    CsrFeat f = f_in;
    // about one unrolled trip per lane for a row of average length
    int lpr = pow2_ceil((int64_t)(f.mean_nnz / kCsrUnroll + 0.5f));
    if (lpr > 4 && (float)(lpr / 2) * kCsrUnroll * 1.1f >= f.mean_nnz) lpr >>= 1;
    lpr = lpr < 4 ? 4 : (lpr > 32 ? 32 : lpr);
    aa_status st = finish_shrink_params(c, sp, choose_tile_rows(c, sp.n_cand, 8.0 * f.mean_nnz + 4.0, 64.0 * 1024));
    if (st != AA_OK) return st;
    void* args[] = {&f, &sp};
    switch (lpr) {
        case 4: return launch_scan(c, score_shrink_csr_kernel<4>, 0, sp, args);
        case 8: return launch_scan(c, score_shrink_csr_kernel<8>, 0, sp, args);
        case 16: return launch_scan(c, score_shrink_csr_kernel<16>, 0, sp, args);
        default: return launch_scan(c, score_shrink_csr_kernel<32>, 0, sp, args);
    }
}

aa_status launch_shrink_from_scores(aa_ctx_impl* c, const float* score, ShrinkParams sp) {
    aa_status st = finish_shrink_params(c, sp, choose_tile_rows(c, sp.n_cand, 4.0, 4.0 * kMaxTileRows));
    if (st != AA_OK) return st;
    void* args[] = {&score, &sp};
    return launch_scan(c, shrink_from_scores_kernel, 0, sp, args);
}

}  // namespace aa

// ---------------------------------------------------------------- shrink + compact without any allocation
// The scan state of this variant (control block + one look-back word per 1024-candidate tile)
// lives in a file-scope device array instead of a caller-provided workspace.  Every device that
// loads the library holds the array until the process exits.
namespace aa {
namespace {

constexpr int64_t kStaticMaxCandidates = AA_STATIC_MAX_CANDIDATES;
constexpr int kStaticTileRows = kMaxTileRows;
constexpr int64_t kStaticMaxTiles = kStaticMaxCandidates / kStaticTileRows;
static_assert(kStaticMaxCandidates % kStaticTileRows == 0, "whole tiles");

struct StaticScan {
    Control ctl;
    unsigned long long tile_state[kStaticMaxTiles];
};

static __device__ __align__(256) unsigned char g_static_scan[sizeof(StaticScan)];

// Host-side record per device: the array's device address (the symbol itself is only a host
// stand-in) and the kernel's resident-CTA count.
struct StaticScanDevice {
    bool ready;
    StaticScan* scan;
    int grid_cap;
};
constexpr int kStaticMaxDevices = 64;
StaticScanDevice g_static_dev[kStaticMaxDevices];
std::mutex g_static_mutex;

aa_status static_scan_for_current_device(StaticScanDevice& out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return AA_ERR_CUDA;
    if (dev < 0 || dev >= kStaticMaxDevices) return AA_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticScanDevice& d = g_static_dev[dev];
    if (!d.ready) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scan) != cudaSuccess || !ptr) return AA_ERR_CUDA;
        int sms = 0, per_sm = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, (const void*)shrink_from_scores_kernel, kScanThreads, 0) != cudaSuccess ||
            per_sm < 1)
            return AA_ERR_CUDA;
        d.scan = static_cast<StaticScan*>(ptr);
        d.grid_cap = per_sm * sms;
        d.ready = true;
    }
    out = d;
    return AA_OK;
}

}  // namespace
}  // namespace aa

extern "C" aa_status aa_shrink_compact_static(const float* score, int64_t n, int64_t id_base, float mix, uint64_t seed,
                                              uint64_t step, int32_t* out_idx, int64_t capacity, int32_t* out_count,
                                              uint8_t* out_mask, int32_t* out_status, void* cuda_stream) {
    using namespace aa;
    if (!out_count || capacity < 0 || (capacity > 0 && !out_idx) || !(mix >= 0.0f && mix <= 1.0f)) return AA_ERR_INVALID_ARG;
    if (n < 0 || (n > 0 && !score)) return AA_ERR_INVALID_ARG;
    if (n > kStaticMaxCandidates) return AA_ERR_WORKSPACE;   // beyond what the built-in scratch array covers
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    StaticScanDevice dev;
    aa_status st = static_scan_for_current_device(dev);
    if (st != AA_OK) return st;
    if (n == 0) {
        if (cudaMemsetAsync(out_count, 0, sizeof(int32_t), stream) != cudaSuccess) return AA_ERR_CUDA;
        if (out_status && cudaMemsetAsync(out_status, 0, sizeof(int32_t), stream) != cudaSuccess) return AA_ERR_CUDA;
        return AA_OK;
    }
    ShrinkParams sp;
    memset(&sp, 0, sizeof sp);
    sp.n_cand = n;
    sp.n_stored = n;
    sp.id_base = id_base;
    sp.mix = mix;
    sp.seed_lo = (uint32_t)seed;
    sp.seed_hi = (uint32_t)(seed >> 32);
    sp.step_lo = (uint32_t)step;
    sp.step_hi = (uint32_t)(step >> 32);
    sp.out_idx = out_idx;
    sp.capacity = capacity;
    sp.out_count = out_count;
    sp.out_mask = out_mask;
    sp.tile_rows = kStaticTileRows;
    sp.n_tiles = (unsigned int)((n + kStaticTileRows - 1) / kStaticTileRows);
    sp.ctl = &dev.scan->ctl;
    sp.tile_state = dev.scan->tile_state;
    // The array keeps whatever the previous call left: ticket, counters, flag generation, status
    // and this call's look-back words all start from zero.
    const size_t used = sizeof(Control) + sizeof(unsigned long long) * sp.n_tiles;
    if (cudaMemsetAsync(dev.scan, 0, used, stream) != cudaSuccess) return AA_ERR_CUDA;
    int grid = dev.grid_cap;
    if ((unsigned int)grid > sp.n_tiles) grid = (int)sp.n_tiles;
    void* args[] = {&score, &sp};
    if (cudaLaunchKernel((const void*)shrink_from_scores_kernel, dim3(grid), dim3(kScanThreads), args, 0, stream) != cudaSuccess)
        return AA_ERR_CUDA;
    if (out_status &&
        cudaMemcpyAsync(out_status, &dev.scan->ctl.status, sizeof(int32_t), cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
        return AA_ERR_CUDA;
    return AA_OK;
}
