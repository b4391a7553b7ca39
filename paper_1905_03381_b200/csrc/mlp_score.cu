// Assistant score -> Bernoulli shrink -> ordered batch list for the two-layer Assistant
//   s_i = w2 . relu(W1 x_i + b1) + b2        (bf16 features and W1, fp32 accumulation),
// where scoring is a dense contraction [candidates x d] * [d x hidden] and runs on the
// tcgen05 tensor cores (Sec. "Learning to generate smart training batches" asks only for a light-weight classifier g; this is the
// library's dense-contraction Assistant).
//
// One persistent CTA per SM, 12 warps (18 when a candidate list selects the rows: warps 3 and 12..17
// then issue row gathers beside warp 0).  A CTA owns super-tiles of 256 candidates: two 128-row
// accumulators [128 x hidden] fp32 side by side in tensor memory, so that every 64-wide K-slice
// of W1 fetched into shared memory is used for 256 candidates.
//   warp 0      : TMA producer.  Per K-slice 256 feature rows x 64 columns (one box, or 64
//                 four-row gathers spread over eight warps when a candidate list selects the rows) and one box of
//                 `hidden` W1 rows x 64 columns (128-byte swizzle) into a 3-stage ring.
//   warp 1      : issues tcgen05.mma (M = 128, N = hidden, K = 16; 8 per stage), commits each
//                 stage back to the producer and the finished super-tile to the epilogue.
//   warp 2      : owns the TMEM allocation; then the tail: Philox keep/skip decisions of
//                 Algorithm 1, ballots, decoupled look-back, ordered append (scan_tail.cuh).
//   warps 4..11 : epilogue.  Each thread reads its candidate's row of pre-activations from TMEM,
//                 applies bias and ReLU and contracts with w2; scores go to the tail through
//                 shared memory and never touch HBM.
// Super-tiles are assigned round-robin (tile = blockIdx.x + k * gridDim.x); the grid never
// exceeds the SM count, so every tile a look-back waits on belongs to a resident CTA.  All
// waits are bounded and give up with AA_ERR_SCAN_TIMEOUT latched.
#include "mlp_pipeline.cuh"
#include "scan_tail.cuh"

namespace aa {

namespace {

constexpr int kMlpThreads = 576;               // with a candidate list: warps 12..17 only help with row gathers
constexpr int kMlpThreadsDense = 384;          // adjacent rows: one box per stage, no helpers
constexpr int kEpiWarps = 8;

struct ScoreControl {
    TilePipe pipe;
    uint64_t s_full[2], s_empty[2];
};

struct MlpKernelParams {
    const float* b1;
    const float* w2;
    const float* b2;
    MlpGeom g;
    uint32_t* gate_out;     // optional [candidates][kMaxHidden / 32]: bit (u & 31) of word u >> 5 = [a_u > 0] of that candidate
};

__device__ __forceinline__ void mlp_give_up(const ShrinkParams& p, TilePipe* tp) {
    latch(p.ctl, AA_ERR_SCAN_TIMEOUT);
    *(volatile int*)&tp->abort_flag = 1;
}

template <bool GATHER>
__global__ void __launch_bounds__(GATHER ? kMlpThreads : kMlpThreadsDense, 1)
mlp_score_shrink_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                        MlpKernelParams mp, ShrinkParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    float* b1_s = reinterpret_cast<float*>(ring + (size_t)kMlpStages * mp.g.stage_bytes);
    float* w2_s = b1_s + kMaxHidden;
    float* s_tile = w2_s + kMaxHidden;                      // [2][kSuperRows]
    ScoreControl* cb = reinterpret_cast<ScoreControl*>(s_tile + 2 * kSuperRows);
    TilePipe* tp = &cb->pipe;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        tile_pipe_init(tp, kEpiWarps);
        for (int q = 0; q < 2; ++q) {
            mbar_init(&cb->s_full[q], kEpiWarps);
            mbar_init(&cb->s_empty[q], 1);
        }
        mbar_fence_init();
        prefetch_tensormap(&map_x);
        prefetch_tensormap(&map_w);
    }
    for (int j = tid; j < kMaxHidden; j += (int)blockDim.x) {
        b1_s[j] = j < mp.g.hidden ? mp.b1[j] : 0.0f;
        w2_s[j] = j < mp.g.hidden ? mp.w2[j] : 0.0f;
    }
    if (warp == 2) tmem_alloc(&tp->tmem_base, kTmemCols);
    const unsigned int epoch = read_epoch(p);
    volatile int* abort_flag = &tp->abort_flag;
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *(volatile uint32_t*)&tp->tmem_base;
    const unsigned int n_tiles = p.n_tiles;

    if (warp == 0) {
        if (!mlp_produce<GATHER>(tp, ring, &map_x, &map_w, mp.g, n_tiles, p.row_idx, p.n_cand, p.n_stored) && lane == 0)
            mlp_give_up(p, tp);
    } else if (GATHER && (warp == 3 || warp >= 12)) {
        if (!mlp_produce<GATHER>(tp, ring, &map_x, &map_w, mp.g, n_tiles, p.row_idx, p.n_cand, p.n_stored, warp == 3 ? 1 : warp - 10) && lane == 0)
            mlp_give_up(p, tp);
    } else if (warp == 1) {
        if (!mlp_issue_mma(tp, ring, mp.g, n_tiles, tmem_base) && lane == 0) mlp_give_up(p, tp);
    } else if (warp == 2) {
        // ------------------------------------------------------------ tail: shrink + ordered append
        int it = 0;
        for (unsigned int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
            const int buf = it & 1;
            if (!mbar_wait(&cb->s_full[buf], (uint32_t)((it >> 1) & 1), abort_flag)) {
                if (lane == 0) mlp_give_up(p, tp);
                break;
            }
            float sv[kSuperRows / 32];
#pragma unroll
            for (int u = 0; u < kSuperRows / 32; ++u) sv[u] = s_tile[buf * kSuperRows + u * 32 + lane];
            __syncwarp();
            if (lane == 0) mbar_arrive(&cb->s_empty[buf]);
            if (GATHER) {
                // a list entry outside the stored rows was scored on a stand-in row: void it (and latch)
#pragma unroll
                for (int u = 0; u < kSuperRows / 32; ++u) {
                    const long long k = (long long)tile * kSuperRows + u * 32 + lane;
                    if (k < p.n_cand && candidate_row(p, k) < 0) sv[u] = __builtin_nanf("");
                }
            }
            warp_shrink_compact<kSuperRows / 32>(p, tile, epoch, kSuperRows / 32, sv);
        }
    } else if (warp >= 4 && warp < 12) {
        // ------------------------------------------------------------ epilogue
        const int quad = warp & 3;                  // TMEM lanes 32*quad .. +31 are this warp's
        const int acc = (warp - 4) >> 2;            // which of the two accumulators
        const int row = acc * 128 + quad * 32 + lane;
        const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * kMaxHidden);
        const float bias2 = *mp.b2;
        int it = 0;
        for (unsigned int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
            const int buf = it & 1;
            if (!mbar_wait(&tp->acc_full[0], (uint32_t)(it & 1), abort_flag) ||
                !mbar_wait(&cb->s_empty[buf], (uint32_t)(((it >> 1) & 1) ^ 1), abort_flag)) {
                if (lane == 0) mlp_give_up(p, tp);
                break;
            }
            tc_fence_after_sync();
            float s = 0.0f;
            uint32_t gate[kMaxHidden / 32];             // this candidate's gates [a_u > 0], one bit per hidden unit
#pragma unroll
            for (int c = 0; c < kMaxHidden / 32; ++c) {
                const int c0 = c * 32;
                gate[c] = 0u;
                if (c0 < mp.g.hidden) {
                    uint32_t r[32];
                    tmem_ld_32cols(t_row + (uint32_t)c0, r);
                    tmem_ld_wait();
                    // hidden is a multiple of 16: the accumulator columns past it were never written and may hold anything
                    if (c0 + 32 > mp.g.hidden) {
#pragma unroll
                        for (int q = 16; q < 32; ++q) r[q] = 0u;
                    }
                    uint32_t bits = 0u;
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const float4 bq = reinterpret_cast<const float4*>(b1_s + c0)[q];
                        const float4 wq = reinterpret_cast<const float4*>(w2_s + c0)[q];
                        const float a0 = __uint_as_float(r[4 * q + 0]) + bq.x, a1 = __uint_as_float(r[4 * q + 1]) + bq.y;
                        const float a2 = __uint_as_float(r[4 * q + 2]) + bq.z, a3 = __uint_as_float(r[4 * q + 3]) + bq.w;
                        s = fmaf(fmaxf(a0, 0.0f), wq.x, s);
                        s = fmaf(fmaxf(a1, 0.0f), wq.y, s);
                        s = fmaf(fmaxf(a2, 0.0f), wq.z, s);
                        s = fmaf(fmaxf(a3, 0.0f), wq.w, s);
                        if (!GATHER)
                            bits |= (a0 > 0.0f ? 1u : 0u) << (4 * q) | (a1 > 0.0f ? 2u : 0u) << (4 * q) | (a2 > 0.0f ? 4u : 0u) << (4 * q) |
                                    (a3 > 0.0f ? 8u : 0u) << (4 * q);
                    }
                    gate[c] = bits;
                }
            }
            s_tile[buf * kSuperRows + row] = s + bias2;
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&tp->acc_empty[0]);
                mbar_arrive(&cb->s_full[buf]);
            }
            // the gates stay behind for an update that follows this screening on the same rows (32 bytes per candidate)
            const long long k = (long long)tile * kSuperRows + row;
            if (!GATHER && mp.gate_out && k < p.n_cand) {
                uint4* dst = reinterpret_cast<uint4*>(mp.gate_out + k * (kMaxHidden / 32));
                dst[0] = make_uint4(gate[0], gate[1], gate[2], gate[3]);
                dst[1] = make_uint4(gate[4], gate[5], gate[6], gate[7]);
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 2) tmem_dealloc(tmem_base, kTmemCols);
    scan_epilogue(p, epoch);
}

}  // namespace

bool encode_bf16_tile_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t row_stride,
                          uint32_t box_rows) {
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
            qres != cudaDriverEntryPointSuccess)
            return false;
        encode = reinterpret_cast<EncodeFn>(fn);
    }
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {row_stride * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

aa_status launch_score_shrink_mlp(aa_ctx_impl* c, const MlpFeat& f, ShrinkParams sp) {
    if (f.hidden < 16 || f.hidden > kMaxHidden || f.hidden % 16) return AA_ERR_UNSUPPORTED;
    if ((uintptr_t)f.x % 16 || (f.row_stride * 2) % 16 || (uintptr_t)f.W1_bf16 % 16 || (f.d * 2) % 16) return AA_ERR_UNSUPPORTED;
    const bool gather = sp.row_idx != nullptr;
    alignas(64) CUtensorMap map_x, map_w;
    if (!encode_bf16_tile_map(&map_x, f.x, (uint64_t)f.n, (uint64_t)f.d, (uint64_t)f.row_stride, gather ? 1 : kSuperRows) ||
        !encode_bf16_tile_map(&map_w, f.W1_bf16, (uint64_t)f.hidden, (uint64_t)f.d, (uint64_t)f.d, (uint32_t)f.hidden))
        return AA_ERR_CUDA;
    MlpKernelParams mp;
    mp.b1 = f.b1;
    mp.w2 = f.w2;
    mp.b2 = f.b2;
    mp.g = make_mlp_geom(f.d, f.hidden);
    aa_status st = finish_shrink_params(c, sp, kSuperRows);
    if (st != AA_OK) return st;
    // Gates of the pool's rows for a later update: only when candidate k is stored row k and the workspace has room.
    const bool keep_gates = !gather && c->mlp_gate_cand && sp.n_cand <= c->max_rows;
    mp.gate_out = keep_gates ? c->mlp_gate_cand : nullptr;
    c->gate_feat = keep_gates ? f.x : nullptr;
    c->gate_w1 = f.W1_bf16;
    c->gate_n = sp.n_cand;
    const size_t smem = 1024 + (size_t)kMlpStages * mp.g.stage_bytes + sizeof(float) * (2 * kMaxHidden + 2 * kSuperRows) +
                        sizeof(ScoreControl) + 64;
    const void* kernel = gather ? (const void*)mlp_score_shrink_kernel<true> : (const void*)mlp_score_shrink_kernel<false>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return AA_ERR_CUDA;
    int grid = c->sm_count;
    if ((unsigned int)grid > sp.n_tiles) grid = (int)sp.n_tiles;
    void* args[] = {&map_x, &map_w, &mp, &sp};
    if (cudaLaunchKernel(kernel, dim3(grid), dim3(gather ? kMlpThreads : kMlpThreadsDense), args, smem, c->stream) != cudaSuccess) return AA_ERR_CUDA;
    ++c->launches;
    return AA_OK;
}

}  // namespace aa
