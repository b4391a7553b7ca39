// Assistant score -> Bernoulli shrink -> ordered batch list for the two-layer Assistant
//   s_i = w2 . relu(W1 x_i + b1) + b2        (bf16 features and W1, fp32 accumulation),
// where scoring is a dense contraction [candidates x d] * [d x hidden] and runs on the
// tcgen05 tensor cores (Sec. 5.2 asks only for a light-weight classifier g; this is the
// library's dense-contraction Assistant).
//
// One persistent CTA per SM, 12 warps.  A CTA owns super-tiles of 256 candidates: two 128-row
// accumulators [128 x hidden] fp32 side by side in tensor memory, so that every 64-wide K-slice
// of W1 fetched into shared memory is used for 256 candidates.
//   warp 0      : TMA producer.  Per K-slice one box of 256 feature rows x 64 columns and one
//                 box of `hidden` W1 rows x 64 columns (128-byte swizzle) into a 3-stage ring.
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
#include "scan_tail.cuh"
#include "tensor_core.cuh"

namespace aa {

namespace {

constexpr int kMlpThreads = 384;
constexpr int kSuperRows = 256;                 // candidates per super-tile (two M = 128 accumulators)
constexpr int kSliceK = 64;                     // bf16 elements per 128-byte swizzled row
constexpr int kMlpStages = 3;
constexpr int kABytes = kSuperRows * 128;       // feature slice of one stage
constexpr int kMaxHidden = 256;
constexpr int kEpiWarps = 8;
constexpr int kTmemCols = 512;

struct MlpControl {
    uint64_t full[kMlpStages], empty[kMlpStages];
    uint64_t acc_full, acc_empty, drain;
    uint64_t s_full[2], s_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

struct MlpKernelParams {
    const float* b1;
    const float* w2;
    const float* b2;
    int hidden;
    int k_slices;          // ceil(d / 64)
    uint32_t b_bytes;      // hidden * 128
    uint32_t stage_bytes;  // kABytes + b_bytes rounded up to 1024
};

__device__ __forceinline__ void mlp_give_up(const ShrinkParams& p, MlpControl* cb) {
    latch(p.ctl, AA_ERR_SCAN_TIMEOUT);
    *(volatile int*)&cb->abort_flag = 1;
}

__global__ void __launch_bounds__(kMlpThreads, 1)
mlp_score_shrink_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                        MlpKernelParams mp, ShrinkParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    float* b1_s = reinterpret_cast<float*>(ring + (size_t)kMlpStages * mp.stage_bytes);
    float* w2_s = b1_s + kMaxHidden;
    float* s_tile = w2_s + kMaxHidden;                      // [2][kSuperRows]
    MlpControl* cb = reinterpret_cast<MlpControl*>(s_tile + 2 * kSuperRows);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kMlpStages; ++s) {
            mbar_init(&cb->full[s], 1);
            mbar_init(&cb->empty[s], 1);
        }
        mbar_init(&cb->acc_full, 1);
        mbar_init(&cb->acc_empty, kEpiWarps);
        mbar_init(&cb->drain, 1);
        for (int q = 0; q < 2; ++q) {
            mbar_init(&cb->s_full[q], kEpiWarps);
            mbar_init(&cb->s_empty[q], 1);
        }
        cb->abort_flag = 0;
        mbar_fence_init();
        prefetch_tensormap(&map_x);
        prefetch_tensormap(&map_w);
    }
    for (int j = tid; j < kMaxHidden; j += kMlpThreads) {
        b1_s[j] = j < mp.hidden ? mp.b1[j] : 0.0f;
        w2_s[j] = j < mp.hidden ? mp.w2[j] : 0.0f;
    }
    if (warp == 2) tmem_alloc(&cb->tmem_base, kTmemCols);
    const unsigned int epoch = read_epoch(p);
    volatile int* abort_flag = &cb->abort_flag;
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *(volatile uint32_t*)&cb->tmem_base;
    const unsigned int n_tiles = p.n_tiles;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        int stage = 0, j = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (unsigned int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
            const int row0 = (int)(tile * (unsigned int)kSuperRows);
            for (int ks = 0; ks < mp.k_slices; ++ks) {
                if (!mbar_wait(&cb->empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                if (lane == 0) {
                    unsigned char* a_dst = ring + (size_t)stage * mp.stage_bytes;
                    mbar_arrive_expect_tx(&cb->full[stage], (uint32_t)kABytes + mp.b_bytes);
                    tma_load_2d(a_dst, &map_x, ks * kSliceK, row0, &cb->full[stage]);
                    tma_load_2d(a_dst + kABytes, &map_w, ks * kSliceK, 0, &cb->full[stage]);
                }
                __syncwarp();
                ++j;
                if (++stage == kMlpStages) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok) {
            if (lane == 0) mlp_give_up(p, cb);
            // let copies still in flight land before the CTA's shared memory goes away
            const int pending = j < kMlpStages ? j : kMlpStages;
            for (int back = 1; back <= pending; ++back) {
                const int jj = j - back, st = jj % kMlpStages, use = jj / kMlpStages;
                const long long t0 = clock64();
                while (!mbar_try_wait(&cb->full[st], (uint32_t)(use & 1)) && clock64() - t0 < kWaitCycles) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        const uint32_t idesc = umma_idesc_bf16(128, mp.hidden, false, false);
        int stage = 0, it = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (unsigned int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++it) {
            // the epilogue has drained both accumulators of the previous super-tile
            if (!mbar_wait(&cb->acc_empty, (uint32_t)((it & 1) ^ 1), abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            for (int ks = 0; ks < mp.k_slices; ++ks) {
                if (!mbar_wait(&cb->full[stage], phase, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                if (lane == 0) {
                    const uint32_t a_addr = smem_u32(ring + (size_t)stage * mp.stage_bytes);
                    const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
                    for (int k = 0; k < kSliceK / 16; ++k) {
                        const uint64_t b_desc = umma_smem_desc(b_addr + k * 32, 16, 1024);
                        const bool acc = (ks | k) != 0;
                        umma_bf16(tmem_base, umma_smem_desc(a_addr + k * 32, 16, 1024), b_desc, idesc, acc);
                        umma_bf16(tmem_base + kMaxHidden, umma_smem_desc(a_addr + 128 * 128 + k * 32, 16, 1024), b_desc, idesc, acc);
                    }
                    umma_commit(&cb->empty[stage]);                               // stage reusable once these MMAs are done
                    if (ks == mp.k_slices - 1) umma_commit(&cb->acc_full);        // super-tile finished
                }
                __syncwarp();
                if (++stage == kMlpStages) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok && lane == 0) mlp_give_up(p, cb);
        // every MMA issued by this thread has retired before the tensor memory is released
        if (lane == 0) umma_commit(&cb->drain);
        __syncwarp();
        {
            const long long t0 = clock64();
            while (!mbar_try_wait(&cb->drain, 0) && clock64() - t0 < kWaitCycles) {}
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------ tail: shrink + ordered append
        int it = 0;
        for (unsigned int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
            const int buf = it & 1;
            if (!mbar_wait(&cb->s_full[buf], (uint32_t)((it >> 1) & 1), abort_flag)) {
                if (lane == 0) mlp_give_up(p, cb);
                break;
            }
            float sv[kSuperRows / 32];
#pragma unroll
            for (int u = 0; u < kSuperRows / 32; ++u) sv[u] = s_tile[buf * kSuperRows + u * 32 + lane];
            __syncwarp();
            if (lane == 0) mbar_arrive(&cb->s_empty[buf]);
            warp_shrink_compact<kSuperRows / 32>(p, tile, epoch, kSuperRows / 32, sv);
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------ epilogue
        const int quad = warp & 3;                  // TMEM lanes 32*quad .. +31 are this warp's
        const int acc = (warp - 4) >> 2;            // which of the two accumulators
        const int row = acc * 128 + quad * 32 + lane;
        const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * kMaxHidden);
        const float bias2 = *mp.b2;
        int it = 0;
        for (unsigned int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
            const int buf = it & 1;
            if (!mbar_wait(&cb->acc_full, (uint32_t)(it & 1), abort_flag) ||
                !mbar_wait(&cb->s_empty[buf], (uint32_t)(((it >> 1) & 1) ^ 1), abort_flag)) {
                if (lane == 0) mlp_give_up(p, cb);
                break;
            }
            tc_fence_after_sync();
            float s = 0.0f;
            for (int c0 = 0; c0 < mp.hidden; c0 += 32) {
                uint32_t r[32];
                tmem_ld_32cols(t_row + (uint32_t)c0, r);
                tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const float4 bq = reinterpret_cast<const float4*>(b1_s + c0)[q];
                    const float4 wq = reinterpret_cast<const float4*>(w2_s + c0)[q];
                    s = fmaf(fmaxf(__uint_as_float(r[4 * q + 0]) + bq.x, 0.0f), wq.x, s);
                    s = fmaf(fmaxf(__uint_as_float(r[4 * q + 1]) + bq.y, 0.0f), wq.y, s);
                    s = fmaf(fmaxf(__uint_as_float(r[4 * q + 2]) + bq.z, 0.0f), wq.z, s);
                    s = fmaf(fmaxf(__uint_as_float(r[4 * q + 3]) + bq.w, 0.0f), wq.w, s);
                }
            }
            s_tile[buf * kSuperRows + row] = s + bias2;
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&cb->acc_empty);
                mbar_arrive(&cb->s_full[buf]);
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
    if (sp.row_idx) return AA_ERR_UNSUPPORTED;   // candidates are the stored rows in order
    if ((uintptr_t)f.x % 16 || (f.row_stride * 2) % 16 || (uintptr_t)f.W1_bf16 % 16 || (f.d * 2) % 16) return AA_ERR_UNSUPPORTED;
    alignas(64) CUtensorMap map_x, map_w;
    if (!encode_bf16_tile_map(&map_x, f.x, (uint64_t)f.n, (uint64_t)f.d, (uint64_t)f.row_stride, kSuperRows) ||
        !encode_bf16_tile_map(&map_w, f.W1_bf16, (uint64_t)f.hidden, (uint64_t)f.d, (uint64_t)f.d, (uint32_t)f.hidden))
        return AA_ERR_CUDA;
    MlpKernelParams mp;
    mp.b1 = f.b1;
    mp.w2 = f.w2;
    mp.b2 = f.b2;
    mp.hidden = (int)f.hidden;
    mp.k_slices = (int)((f.d + kSliceK - 1) / kSliceK);
    mp.b_bytes = (uint32_t)f.hidden * 128u;
    mp.stage_bytes = ((uint32_t)kABytes + mp.b_bytes + 1023u) & ~1023u;
    aa_status st = finish_shrink_params(c, sp, kSuperRows);
    if (st != AA_OK) return st;
    const size_t smem = 1024 + (size_t)kMlpStages * mp.stage_bytes + sizeof(float) * (2 * kMaxHidden + 2 * kSuperRows) +
                        sizeof(MlpControl) + 64;
    const void* kernel = (const void*)mlp_score_shrink_kernel;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return AA_ERR_CUDA;
    int grid = c->sm_count;
    if ((unsigned int)grid > sp.n_tiles) grid = (int)sp.n_tiles;
    void* args[] = {&map_x, &map_w, &mp, &sp};
    if (cudaLaunchKernel(kernel, dim3(grid), dim3(kMlpThreads), args, smem, c->stream) != cudaSuccess) return AA_ERR_CUDA;
    ++c->launches;
    return AA_OK;
}

}  // namespace aa
