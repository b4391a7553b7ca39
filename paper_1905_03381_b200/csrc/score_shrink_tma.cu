// Assistant score -> Bernoulli shrink -> ordered batch list for 16-byte aligned dense rows,
// as two persistent, warp-specialised CTAs per SM fed by bulk asynchronous copies (one CTA's start-up and tail then
// overlap the other's streaming; together their rings hold as many bytes in flight as one CTA's ring of twice the depth).
//
//   producer warp : starts on tile blockIdx.x, then takes tile tickets (the next one is requested
//                   a few stages before the current tile ends) and streams the tile's rows into a shared-memory ring with
//                   cp.async.bulk (one copy per stage of contiguous rows, or one per row when a
//                   candidate list gathers rows); it runs ahead of the consumers by the depth of
//                   the ring, across tile boundaries.  Its per-stage work is a handful of
//                   instructions: stage index and phase are running counters.
//   consumer warps: `split` warps share each stage (disjoint rows): dot products with the
//                   Assistant weights (shared memory, conflict-free layout), pre-activations
//                   into a small score ring.  Stage and score slot follow from the stage
//                   sequence number, so no per-stage record is exchanged.
//   tail warps    : per finished tile, the Philox keep/skip decisions of Algorithm 1, warp
//                   ballots, the decoupled look-back and the ordered append (scan_tail.cuh).
//                   A look-back costs several L2 round trips, so consecutive tiles go to
//                   different tail warps and their look-backs overlap.
//
// The roles meet only through mbarriers (full/empty per ring stage and per score slot); every
// wait is bounded and, on giving up, latches AA_ERR_SCAN_TIMEOUT, raises the CTA's abort flag
// and lets all roles drain and return.
#include "async_copy.cuh"
#include "scan_tail.cuh"

namespace aa {

namespace {

constexpr int kMaxRowBytes = 24 * 1024;              // longest row the ring takes
constexpr int kTargetStage = 32 * 1024;              // preferred bytes of one ring stage
constexpr int kMaxStages = 4;
constexpr int kMaxSplit = 2;                         // consumer warps per stage
constexpr int kConsumers = kMaxStages * kMaxSplit;
constexpr int kTails = 2;                            // tail warps: tile q goes to tail q % kTails
constexpr int kTmaThreads = (kConsumers + 1 + kTails) * 32;   // warp 0 producer, 1..8 consumers, 9..10 tails
constexpr int kSlotShift = 3;
constexpr int kScoreSlots = 1 << kSlotShift;         // tiles in flight between consumers and tails
constexpr int kMaxUnits = 8;                         // 32-candidate units per tile

struct TmaGeometry {
    int chunk_rows;        // rows per ring stage (power of two <= 32)
    int cpt_shift;         // log2(chunks per tile)
    int stages;
    int stage_bytes;       // bytes reserved per stage (a multiple of 128)
    int split;             // consumer warps sharing one stage (1 or 2)
    int contiguous;        // rows of a chunk are adjacent in memory: one copy per chunk
    int nvec;              // 16-byte vectors per row
    int slot_rows;         // floats reserved per score slot (tile rows rounded up to a warp)
    uint32_t row_bytes;
};

struct RingControl {
    uint64_t x_full[kMaxStages], x_empty[kMaxStages];
    uint64_t s_full[kScoreSlots], s_empty[kScoreSlots];
    unsigned int tile_of_slot[kScoreSlots];
    int stop_j;            // first stage sequence number that carries no data
    int stop_q;            // first tile sequence number that carries no data
    int abort_flag;
};

__device__ __forceinline__ void give_up(const ShrinkParams& p, RingControl* cb) {
    latch(p.ctl, AA_ERR_SCAN_TIMEOUT);
    *(volatile int*)&cb->abort_flag = 1;
}

// Dot products of `rows` staged rows (row_bytes apart).  LPR lanes per row.
template <typename T, int LPR>
__device__ __forceinline__ void consume_rows(const unsigned char* xs, const float* w_s, int rows, int nvec,
                                             uint32_t row_bytes, float bias, float* s_out, int lane) {
    constexpr int VE = Vec<T>::kElems;
    if (LPR == 32) {
        int i = 0;
        for (; i + 1 < rows; i += 2) {   // two rows share every weight read
            const uint4* r0 = reinterpret_cast<const uint4*>(xs + (size_t)i * row_bytes);
            const uint4* r1 = reinterpret_cast<const uint4*>(xs + (size_t)(i + 1) * row_bytes);
            float p0[VE], p1[VE];   // one partial sum per vector element: independent FMA chains
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
            float a0 = 0.0f, a1 = 0.0f;
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
            if (lane == 0) {
                s_out[i] = a0 + bias;
                s_out[i + 1] = a1 + bias;
            }
        }
        if (i < rows) {
            const uint4* r0 = reinterpret_cast<const uint4*>(xs + (size_t)i * row_bytes);
            float p0[VE];
#pragma unroll
            for (int e = 0; e < VE; ++e) p0[e] = 0.0f;
#pragma unroll 4
            for (int v = lane; v < nvec; v += 32) {
                float x0[VE], wq[VE];
                Vec<T>::unpack(r0[v], x0);
                Vec<T>::load_w(w_s, nvec, v, wq);
#pragma unroll
                for (int e = 0; e < VE; ++e) p0[e] = fmaf(x0[e], wq[e], p0[e]);
            }
            float a0 = 0.0f;
#pragma unroll
            for (int e = 0; e < VE; ++e) a0 += p0[e];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a0 += __shfl_xor_sync(0xFFFFFFFFu, a0, o);
            if (lane == 0) s_out[i] = a0 + bias;
        }
    } else {
        constexpr int G = 32 / LPR;
        const int grp = lane / LPR, gl = lane % LPR;
        for (int i = grp; i < rows; i += G) {   // rows is a multiple of G: every lane runs the same trips
            const uint4* r0 = reinterpret_cast<const uint4*>(xs + (size_t)i * row_bytes);
            float p0[VE];
#pragma unroll
            for (int e = 0; e < VE; ++e) p0[e] = 0.0f;
#pragma unroll 2
            for (int v = gl; v < nvec; v += LPR) {
                float x0[VE], wq[VE];
                Vec<T>::unpack(r0[v], x0);
                Vec<T>::load_w(w_s, nvec, v, wq);
#pragma unroll
                for (int e = 0; e < VE; ++e) p0[e] = fmaf(x0[e], wq[e], p0[e]);
            }
            float a0 = 0.0f;
#pragma unroll
            for (int e = 0; e < VE; ++e) a0 += p0[e];
#pragma unroll
            for (int o = LPR / 2; o > 0; o >>= 1) a0 += __shfl_xor_sync(0xFFFFFFFFu, a0, o);
            if (gl == 0) s_out[i] = a0 + bias;
        }
    }
}

template <typename T, int LPR>
__global__ void __launch_bounds__(kTmaThreads, 2) score_shrink_tma_kernel(DenseFeat f, ShrinkParams p, TmaGeometry g) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int VE = Vec<T>::kElems;
    unsigned char* x_ring = smem;
    float* w_s = reinterpret_cast<float*>(smem + (size_t)g.stages * g.stage_bytes);
    float* s_ring = w_s + (size_t)g.nvec * VE;
    RingControl* cb = reinterpret_cast<RingControl*>(s_ring + kScoreSlots * g.slot_rows);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cpt = 1 << g.cpt_shift;   // chunks (ring stages' worth of rows) per tile
    if (tid == 0) {
        for (int s = 0; s < g.stages; ++s) {
            mbar_init(&cb->x_full[s], 1);
            mbar_init(&cb->x_empty[s], (uint32_t)g.split);
        }
        for (int q = 0; q < kScoreSlots; ++q) {
            mbar_init(&cb->s_full[q], (uint32_t)(cpt * g.split));
            mbar_init(&cb->s_empty[q], 1);
        }
        cb->stop_j = 0x7FFFFFFF;
        cb->stop_q = 0x7FFFFFFF;
        cb->abort_flag = 0;
        mbar_fence_init();
    }
    volatile int* abort_flag = &cb->abort_flag;
    __syncthreads();   // barriers are initialised
    // everything above overlapped the previous kernel's tail; from here on its results are read (weights, scan state)
    grid_dependency_wait();
    grid_dependency_release();
    const float bias = *f.b;
    const unsigned int epoch = read_epoch(p);
    // The consumer warps stage the weights among themselves (named barrier 1) while the
    // producer is already streaming rows.
    if (warp >= 1 && warp <= kConsumers) {
        for (int j = tid - 32; j < f.d; j += kConsumers * 32) w_s[Vec<T>::w_index(j, g.nvec)] = f.w[j];
        asm volatile("bar.sync 1, %0;" ::"n"(kConsumers * 32) : "memory");
    }

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        const unsigned char* base = static_cast<const unsigned char*>(f.base);
        const size_t stride_bytes = (size_t)f.row_stride * sizeof(T);
        const uint32_t chunk_bytes = (uint32_t)g.chunk_rows * g.row_bytes;
        int j = 0, q = 0, stage = 0;
        uint32_t phase = 0;   // parity of the current pass over the ring
        bool ok = true;
        // The first tile of a CTA is its block index (no round trip before the first copy); later
        // tiles come from the ticket counter, which therefore counts from gridDim.x.  The next ticket
        // is requested only a few stages before this tile's last copy is issued, just early enough to
        // hide the atomic: a CTA never holds more than the tile it is streaming, which keeps the
        // CTAs' finishing times close together.
        const int req_c = cpt > 3 ? cpt - 3 : 0;
        unsigned int next_tile = blockIdx.x;
        while (ok) {
            const unsigned int tile = next_tile;
            if (tile >= p.n_tiles) break;
            const int slot = q & (kScoreSlots - 1);
            // the tail has released this score slot (it also guards the slot's tile record)
            if (q >= kScoreSlots && !mbar_wait(&cb->s_empty[slot], (uint32_t)(((q >> kSlotShift) - 1) & 1), abort_flag)) { ok = false; break; }
            if (lane == 0) cb->tile_of_slot[slot] = tile;
            const long long k_tile = (long long)tile * p.tile_rows;
            long long rows_left = p.n_cand - k_tile;   // > 0
            const unsigned char* src = base + (size_t)k_tile * stride_bytes;
            for (int c = 0; c < cpt; ++c) {
                if (c == req_c && lane == 0) next_tile = gridDim.x + atomicAdd(&p.ctl->ticket, 1u);
                if (j >= g.stages && !mbar_wait(&cb->x_empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                unsigned char* dst = x_ring + (size_t)stage * g.stage_bytes;
                if (g.contiguous) {
                    if (lane == 0) {
                        if (rows_left >= g.chunk_rows) {
                            mbar_arrive_expect_tx(&cb->x_full[stage], chunk_bytes);
                            bulk_g2s(dst, src, chunk_bytes, &cb->x_full[stage]);
                        } else if (rows_left > 0) {
                            const uint32_t bytes = (uint32_t)rows_left * g.row_bytes;
                            mbar_arrive_expect_tx(&cb->x_full[stage], bytes);
                            bulk_g2s(dst, src, bytes, &cb->x_full[stage]);
                        } else {
                            mbar_arrive(&cb->x_full[stage]);
                        }
                    }
                    src += chunk_bytes;
                } else {
                    // lane i fetches row i of the chunk
                    long long r = -1;
                    if (lane < g.chunk_rows && lane < rows_left) r = candidate_row(p, k_tile + (long long)c * g.chunk_rows + lane);
                    const unsigned int have = __ballot_sync(0xFFFFFFFFu, r >= 0);
                    if (lane == 0) {
                        if (have) mbar_arrive_expect_tx(&cb->x_full[stage], (uint32_t)__popc(have) * g.row_bytes);
                        else mbar_arrive(&cb->x_full[stage]);
                    }
                    __syncwarp();
                    if (r >= 0) bulk_g2s(dst + (size_t)lane * g.row_bytes, base + (size_t)r * stride_bytes, g.row_bytes, &cb->x_full[stage]);
                }
                rows_left -= g.chunk_rows;
                ++j;
                if (++stage == g.stages) { stage = 0; phase ^= 1u; }
            }
            ++q;
            next_tile = __shfl_sync(0xFFFFFFFFu, next_tile, 0);
        }
        if (ok) {
            // wake every consumer once with an empty stage, then the tail with an empty tile
            if (lane == 0) *(volatile int*)&cb->stop_j = j;
            for (int c = 0; c < g.stages && ok; ++c) {
                if (j >= g.stages && !mbar_wait(&cb->x_empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                if (lane == 0) mbar_arrive(&cb->x_full[stage]);
                ++j;
                if (++stage == g.stages) { stage = 0; phase ^= 1u; }
            }
        }
        if (ok) {
            if (lane == 0) *(volatile int*)&cb->stop_q = q;
            for (int t = 0; t < kTails && ok; ++t, ++q) {
                const int slot = q & (kScoreSlots - 1);
                if (q >= kScoreSlots && !mbar_wait(&cb->s_empty[slot], (uint32_t)(((q >> kSlotShift) - 1) & 1), abort_flag)) { ok = false; break; }
                if (lane == 0)
                    for (int c = 0; c < cpt * g.split; ++c) mbar_arrive(&cb->s_full[slot]);
            }
        }
        if (!ok) {
            if (lane == 0) give_up(p, cb);
            // let copies still in flight land before the CTA's shared memory goes away
            const int pending = j < g.stages ? j : g.stages;
            for (int back = 1; back <= pending; ++back) {
                const int jj = j - back, st = jj % g.stages, use = jj / g.stages;
                const long long t0 = clock64();
                while (!mbar_try_wait(&cb->x_full[st], (uint32_t)(use & 1)) && clock64() - t0 < kWaitCycles) {}
            }
        }
    } else if (warp <= kConsumers) {
        // ------------------------------------------------------------ consumers
        const int cidx = warp - 1;
        const int stage = cidx / g.split, part = cidx - stage * g.split;
        if (stage < g.stages) {
            const int rows_per = g.chunk_rows / g.split;
            const unsigned char* xs = x_ring + (size_t)stage * g.stage_bytes + (size_t)part * rows_per * g.row_bytes;
            for (int n = 0;; ++n) {
                if (!mbar_wait(&cb->x_full[stage], (uint32_t)(n & 1), abort_flag)) {
                    if (lane == 0) give_up(p, cb);
                    break;
                }
                const int j = n * g.stages + stage;
                if (j >= *(volatile int*)&cb->stop_j) break;
                const int chunk = j & (cpt - 1), slot = (j >> g.cpt_shift) & (kScoreSlots - 1);
                consume_rows<T, LPR>(xs, w_s, rows_per, g.nvec, g.row_bytes, bias,
                                     s_ring + slot * g.slot_rows + chunk * g.chunk_rows + part * rows_per, lane);
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(&cb->s_full[slot]);
                    mbar_arrive(&cb->x_empty[stage]);
                }
            }
        }
    } else {
        // ------------------------------------------------------------ tail
        const int units = (p.tile_rows + 31) >> 5;
        for (int q = warp - (kConsumers + 1);; q += kTails) {
            const int slot = q & (kScoreSlots - 1);
            if (!mbar_wait(&cb->s_full[slot], (uint32_t)((q >> kSlotShift) & 1), abort_flag)) {
                if (lane == 0) give_up(p, cb);
                break;
            }
            if (q >= *(volatile int*)&cb->stop_q) break;
            const unsigned int tile = cb->tile_of_slot[slot];
            float sv[kMaxUnits];
#pragma unroll
            for (int u = 0; u < kMaxUnits; ++u) sv[u] = u < units ? s_ring[slot * g.slot_rows + u * 32 + lane] : 0.0f;
            if (p.row_idx && p.out_score) {
                // a candidate whose list entry points outside the store was never copied: its score slot holds stale sums
#pragma unroll
                for (int u = 0; u < kMaxUnits; ++u) {
                    const long long k = (long long)tile * p.tile_rows + u * 32 + lane;
                    if (u < units && k < p.n_cand && (unsigned long long)(long long)p.row_idx[k] >= (unsigned long long)p.n_stored)
                        sv[u] = __int_as_float(0x7FC00000);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&cb->s_empty[slot]);
            warp_shrink_compact<kMaxUnits>(p, tile, epoch, units, sv);
        }
    }
    __syncthreads();
    scan_epilogue(p, epoch);
}

int pow2_floor(int64_t v) {
    int p = 1;
    while ((int64_t)p * 2 <= v) p <<= 1;
    return p;
}

template <typename T>
const void* pick_kernel(int lpr) {
    switch (lpr) {
        case 4: return (const void*)score_shrink_tma_kernel<T, 4>;
        case 8: return (const void*)score_shrink_tma_kernel<T, 8>;
        case 16: return (const void*)score_shrink_tma_kernel<T, 16>;
        default: return (const void*)score_shrink_tma_kernel<T, 32>;
    }
}

}  // namespace

aa_status launch_score_shrink_dense_tma(aa_ctx_impl* c, const DenseFeat& f_in, ShrinkParams sp) {
    DenseFeat f = f_in;
    const int es = f.dtype == AA_BF16 ? 2 : 4;
    const int ve = 16 / es;
    const int64_t row_bytes = f.d * es;
    if (row_bytes > kMaxRowBytes || row_bytes < 256) return AA_ERR_UNSUPPORTED;   // tiny rows: the load-based kernel does well
    TmaGeometry g;
    g.row_bytes = (uint32_t)row_bytes;
    g.nvec = (int)(f.d / ve);
    g.chunk_rows = pow2_floor(kTargetStage / row_bytes);
    if (g.chunk_rows > 32) g.chunk_rows = 32;
    g.stage_bytes = (int)(((int64_t)g.chunk_rows * row_bytes + 127) / 128 * 128);
    g.split = g.chunk_rows >= 2 ? kMaxSplit : 1;
    g.contiguous = (!sp.row_idx && f.row_stride == f.d) ? 1 : 0;
    const int rows_per = g.chunk_rows / g.split;

    int lpr = 1;
    while (lpr < 32 && lpr * 2 <= g.nvec) lpr <<= 1;   // at least two vectors per lane when rows are short
    if (lpr > 1 && g.nvec < 64) lpr >>= 1;
    if (lpr < 4) lpr = 4;
    if (32 / lpr > rows_per) lpr = 32 / rows_per;

    // tile = one look-back unit and one ticket: enough rows for ~128 KB, at least 32, a multiple of the
    // chunk.  (Shorter tiles would even out the CTAs' finishing times, but the look-back then costs more
    // than it saves: 16-row tiles measured 10 % slower at 65,536 x 3072 bf16.)
    int units = 1;
    while (units < kMaxUnits && (int64_t)units * 32 * row_bytes < 128 * 1024) units <<= 1;
    while (units > 1 && sp.n_cand / (units * 32) < 4 * (int64_t)c->sm_count) units >>= 1;
    const int tile_rows = units * 32;
    const int cpt = tile_rows / g.chunk_rows;
    g.cpt_shift = 0;
    while ((1 << g.cpt_shift) < cpt) ++g.cpt_shift;

    g.slot_rows = (tile_rows + 31) / 32 * 32;
    const size_t fixed = (size_t)g.nvec * ve * sizeof(float) + sizeof(float) * kScoreSlots * g.slot_rows + sizeof(RingControl) + 128;
    const size_t budget = 110 * 1024;                  // two CTAs per SM
    if (fixed + 2 * (size_t)g.stage_bytes > budget) return AA_ERR_UNSUPPORTED;
    int stages = (int)((budget - fixed) / g.stage_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    g.stages = stages;
    const size_t smem = fixed + (size_t)stages * g.stage_bytes;

    aa_status st = finish_shrink_params(c, sp, tile_rows);
    if (st != AA_OK) return st;
    const void* kernel = f.dtype == AA_BF16 ? pick_kernel<uint16_t>(lpr) : pick_kernel<float>(lpr);
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return AA_ERR_CUDA;
    int grid = resident_ctas(c, kernel, kTmaThreads, smem);     // two per SM; every CTA's first tile is its block index, so all must be resident
    if (grid <= 0) return AA_ERR_CUDA;
    if ((unsigned int)grid > sp.n_tiles) grid = (int)sp.n_tiles;
    void* args[] = {&f, &sp, &g};
    if (launch_overlapped(c, kernel, dim3(grid), dim3(kTmaThreads), args, smem, false) != cudaSuccess) return AA_ERR_CUDA;
    ++c->launches;
    return AA_OK;
}

}  // namespace aa
