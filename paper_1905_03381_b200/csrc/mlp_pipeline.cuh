// Producer / MMA halves of the two-layer Assistant's first layer, shared by the scoring kernel
// and by the gradient kernel's forward pass:  pre-activations [256 rows x hidden] = X_tile W1^T
// for one super-tile of 256 rows at a time, two 128-row fp32 accumulators side by side in TMEM.
//
//   producer warp : per 64-wide K-slice, 256 feature rows x 64 columns and `hidden` W1 rows x 64
//                   columns (128-byte swizzle) into a 3-stage ring (the gradient's forward pass: 128
//                   rows per tile, 4 stages, the two accumulators alternating between tiles).  Rows come as one TMA box
//                   when the tile's rows are adjacent in memory, or as 64 four-row gathers
//                   (tile::gather4, spread over eight warps) when a row list selects them.
//   MMA warp      : tcgen05.mma M = 128, N = hidden, K = 16, eight per stage; commits every
//                   stage back to the producer and every finished super-tile to `acc_full`.
// The consumer of the accumulators arrives `acc_consumers` times on `acc_empty` per super-tile.
// Every wait is bounded; a role that gives up sets the abort flag and the caller latches the error.
#pragma once

#include "aa_internal.cuh"
#include "tensor_core.cuh"

namespace aa {

constexpr int kSuperRows = 256;                 // rows per super-tile (two M = 128 accumulators)
constexpr int kSliceK = 64;                     // bf16 elements per 128-byte swizzled row
constexpr int kMlpStages = 3;
constexpr int kMaxMlpStages = 4;
constexpr int kHalfRows = 128;                  // rows per tile when two accumulators alternate (one M = 128 accumulator each)
constexpr int kHalfStages = 4;
constexpr int kABytes = kSuperRows * 128;       // feature slice of one stage
constexpr int kMaxHidden = 256;
constexpr int kTmemCols = 512;
constexpr int kGatherWarps = 8;                 // warps that issue the row gathers when a row list selects the rows

struct MlpGeom {
    int hidden;
    int k_slices;          // ceil(d / 64)
    uint32_t b_bytes;      // hidden * 128
    uint32_t stage_bytes;  // kABytes + b_bytes rounded up to 1024
};

struct TilePipe {
    uint64_t full[kMaxMlpStages], empty[kMaxMlpStages];
    uint64_t acc_full[2], acc_empty[2], drain;   // 256-row super-tiles use entry 0; 128-row tiles alternate between the two
    uint32_t tmem_base;
    int abort_flag;
};

inline MlpGeom make_mlp_geom(int64_t d, int64_t hidden, int tile_rows = kSuperRows) {
    MlpGeom g;
    g.hidden = (int)hidden;
    g.k_slices = (int)((d + kSliceK - 1) / kSliceK);
    g.b_bytes = (uint32_t)hidden * 128u;
    g.stage_bytes = ((uint32_t)tile_rows * 128u + g.b_bytes + 1023u) & ~1023u;
    return g;
}

#ifdef __CUDACC__

// Four rows of 64 columns each (the tensor map's box is [1 x 64]) into four consecutive
// 128-byte rows at dst.  x * 2 bytes must be a multiple of 16.
__device__ __forceinline__ void tma_gather4(void* dst, const CUtensorMap* map, int x, int r0, int r1, int r2, int r3, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];" ::"r"(
            smem_u32(dst)),
        "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
        : "memory");
}

__device__ __forceinline__ void tile_pipe_init(TilePipe* tp, uint32_t acc_consumers) {
    for (int s = 0; s < kMaxMlpStages; ++s) {
        mbar_init(&tp->full[s], 1);
        mbar_init(&tp->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
        mbar_init(&tp->acc_full[b], 1);
        mbar_init(&tp->acc_empty[b], acc_consumers);
    }
    mbar_init(&tp->drain, 1);
    tp->abort_flag = 0;
}

// Whole warp.  Tiles of ROWS rows: blockIdx.x, blockIdx.x + gridDim.x, ... below n_tiles.  rows: nullptr = tile t
// holds stored rows [ROWS t, ROWS t + ROWS) (the feature map's box is ROWS rows high); otherwise row k of the list (k < n_list) names the
// stored row, entries outside [0, n_stored) or past the list read row 0 (their results are
// discarded by the consumer).  Returns false if a wait gave up.
template <bool GATHER, int ROWS = kSuperRows, int STAGES = kMlpStages>
__device__ __forceinline__ bool mlp_produce(TilePipe* tp, unsigned char* ring, const CUtensorMap* map_x, const CUtensorMap* map_w,
                                            const MlpGeom& g, unsigned int n_tiles, const int32_t* rows, long long n_list,
                                            long long n_stored, int part = 0) {
    // Gathered rows are fetched by kGatherWarps warps (part = 0 .. kGatherWarps - 1), ROWS / kGatherWarps rows each, one four-row
    // gather per issuing lane and stage: the gathers a single warp issues retire at only about one per 43 ns.  Part 0 is the
    // producer proper (it also posts the expected bytes and loads W1); the others follow the same barriers.
    const int lane = threadIdx.x & 31;
    const bool helper = part != 0;
    volatile int* abort_flag = &tp->abort_flag;
    int stage = 0, j = 0;
    uint32_t phase = 0;
    bool ok = true;
    constexpr int kRowsPerPart = ROWS / kGatherWarps;
    constexpr uint32_t kTileBytes = (uint32_t)ROWS * 128u;
    const bool gather_lane = lane < kRowsPerPart / 4;
    for (unsigned int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const long long k0 = (long long)tile * ROWS;
        int r[4] = {0, 0, 0, 0};
        if (GATHER && gather_lane) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const long long k = k0 + part * kRowsPerPart + lane * 4 + q;
                long long row = k < n_list ? (long long)rows[k] : 0;
                if ((unsigned long long)row >= (unsigned long long)n_stored) row = 0;
                r[q] = (int)row;
            }
        }
        for (int ks = 0; ks < g.k_slices; ++ks) {
            if (!mbar_wait(&tp->empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
            unsigned char* a_dst = ring + (size_t)stage * g.stage_bytes;
            if (lane == 0 && !helper) {
                mbar_arrive_expect_tx(&tp->full[stage], kTileBytes + g.b_bytes);
                tma_load_2d(a_dst + kTileBytes, map_w, ks * kSliceK, 0, &tp->full[stage]);
                if (!GATHER) tma_load_2d(a_dst, map_x, ks * kSliceK, (int)k0, &tp->full[stage]);
            }
            if (GATHER) {
                __syncwarp();
                if (gather_lane)
                    tma_gather4(a_dst + (part * kRowsPerPart + lane * 4) * 128, map_x, ks * kSliceK, r[0], r[1], r[2], r[3], &tp->full[stage]);
            }
            __syncwarp();
            ++j;
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
    }
    if (!ok) {
        // let copies still in flight land before the CTA's shared memory goes away
        const int pending = j < STAGES ? j : STAGES;
        for (int back = 1; back <= pending; ++back) {
            const int jj = j - back, st = jj % STAGES, use = jj / STAGES;
            const long long t0 = clock64();
            while (!mbar_try_wait(&tp->full[st], (uint32_t)(use & 1)) && clock64() - t0 < kWaitCycles) {}
        }
    }
    return ok;
}

// Whole warp; lane 0 issues.  Returns false if a wait gave up.  On return every MMA issued here has retired.
// ROWS = 256: both accumulators hold one super-tile (the consumer drains them before the next one starts).
// ROWS = 128: tile `it` of this CTA accumulates into accumulator it & 1, so the consumer of one tile overlaps
// the products of the next.
template <int ROWS = kSuperRows, int STAGES = kMlpStages>
__device__ __forceinline__ bool mlp_issue_mma(TilePipe* tp, unsigned char* ring, const MlpGeom& g, unsigned int n_tiles, uint32_t tmem_base) {
    const int lane = threadIdx.x & 31;
    volatile int* abort_flag = &tp->abort_flag;
    const uint32_t idesc = umma_idesc_bf16(128, g.hidden, false, false);
    constexpr uint32_t kTileBytes = (uint32_t)ROWS * 128u;
    int stage = 0, it = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (unsigned int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++it) {
        // the consumer has drained the accumulator(s) this tile writes
        const int buf = ROWS == kSuperRows ? 0 : (it & 1);
        const int use = ROWS == kSuperRows ? it : (it >> 1);
        if (!mbar_wait(&tp->acc_empty[buf], (uint32_t)((use & 1) ^ 1), abort_flag)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t acc_addr = tmem_base + (uint32_t)(buf * kMaxHidden);
        for (int ks = 0; ks < g.k_slices; ++ks) {
            if (!mbar_wait(&tp->full[stage], phase, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t a_addr = smem_u32(ring + (size_t)stage * g.stage_bytes);
                const uint32_t b_addr = a_addr + kTileBytes;
#pragma unroll
                for (int k = 0; k < kSliceK / 16; ++k) {
                    const uint64_t b_desc = umma_smem_desc(b_addr + k * 32, 16, 1024);
                    const bool acc = (ks | k) != 0;
                    umma_bf16(acc_addr, umma_smem_desc(a_addr + k * 32, 16, 1024), b_desc, idesc, acc);
                    if (ROWS == kSuperRows)
                        umma_bf16(acc_addr + kMaxHidden, umma_smem_desc(a_addr + 128 * 128 + k * 32, 16, 1024), b_desc, idesc, acc);
                }
                umma_commit(&tp->empty[stage]);                                 // stage reusable once these MMAs are done
                if (ks == g.k_slices - 1) umma_commit(&tp->acc_full[buf]);      // tile finished
            }
            __syncwarp();
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
    }
    if (lane == 0) umma_commit(&tp->drain);
    __syncwarp();
    const long long t0 = clock64();
    while (!mbar_try_wait(&tp->drain, 0) && clock64() - t0 < kWaitCycles) {}
    return ok;
}

#endif  // __CUDACC__

}  // namespace aa
