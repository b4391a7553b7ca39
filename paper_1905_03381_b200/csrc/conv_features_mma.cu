// Features of the convolutional Assistant for bf16 images, on the matrix instructions
// (Sec. "Learning to generate smart training batches", closing paragraph: convolution shared with the Boss -> pooling ->
// single linear layer; this kernel is the convolution, the rectifier and the average pooling).
//
// Per image the convolution is a small dense contraction: [channels x taps] * [taps x pixels] with taps = c_in * k * k
// (27 for a 3 x 3 window over 3 planes) and up to 16 channels.  A warp takes 16 adjacent pixels of an image row at a time,
// as two products of shape 16 channels x 8 pixels x 16 taps (mma.sync.m16n8k16, fp32 accumulation):
//   left operand  (16 channels x 16 taps): the taps, fp32 split into three bf16 terms hi + mid + lo (exact: 3 x 8
//                 significant bits), held in registers for the whole kernel; the three products go into one accumulator (which starts from zero: the bias
//                 enters with the rectifier, max(a, 0) = max(a - bias, -bias) + bias)
//   right operand (16 taps x 8 pixels): one ldmatrix.x2.trans.  Row k of that matrix is tap k's view of the 8 pixels:
//                 8 adjacent elements of the image in shared memory, starting dx elements to the right of the pixels.
//                 ldmatrix wants every row 16-byte aligned, so the image is kept k times, copy dx shifted left by dx
//                 elements; tap (ci, dy, dx) then reads copy dx at an aligned address.
// bf16 x bf16 products are exact in fp32, so the arithmetic is that of an fp32 multiply-add loop up to summation order.
// The rectifier and the pooling work on the accumulator fragments: a thread holds two adjacent pixels of two channels,
// so the window's rows are a running sum over the image rows a warp walks through and its columns an add and at most
// two lane shuffles at the end.
//
// Shapes it does not cover (fp32 images, more than 32 taps or 16 channels, widths that are not a multiple of 16, pooling
// sides other than 1, 2, 4, 8, 16) stay with the per-thread multiply-add kernel (conv_features.cu).
#include <cuda_bf16.h>

#include <mutex>

#include "aa_internal.cuh"
#include "async_copy.cuh"

namespace aa {

namespace {

constexpr int kCmThreads = 128;
constexpr int kCmWarps = kCmThreads / 32;
constexpr int kCmMaxTaps = 32;
constexpr int kCmMaxChan = 16;

struct FastDivM {      // n / d for n * d < 2^32 by one multiply-high (d = 1: magic 0)
    uint32_t d, magic;
    __host__ void set(uint32_t divisor) {
        d = divisor;
        magic = divisor <= 1 ? 0u : (uint32_t)((1ull << 32) / divisor + 1ull);
    }
    __device__ __forceinline__ void divmod(uint32_t n, uint32_t& q, uint32_t& r) const {
        q = magic ? __umulhi(n, magic) : n;
        r = n - q * d;
    }
};

struct ConvMmaParams {
    const uint16_t* x;
    int64_t n, row_stride;
    int c_in, height, width, c_out, ksize, pool;
    const float* weight;     // [c_out][c_in][k][k]
    const float* bias;       // [c_out] or nullptr
    float* phi;
    int64_t phi_stride;
    int wp, hp;              // padded row pitch (elements, a multiple of 8) and padded height of the image in shared memory
    int plane;               // elements per image plane (a multiple of 8, >= hp * wp)
    int copy;                // elements per shifted copy of the image (a multiple of 8, >= c_in * plane)
    int taps;
    int n_vec;               // 16-byte vectors per image
    FastDivM by_pixels, by_width, by_strips;
};

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// the first product of an accumulator: no addend
__device__ __forceinline__ void mma_bf16_16816_first(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%10, %10, %10, %10};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.0f));
}
// Two 8 x 8 matrices of 16-bit elements, transposed on the way: lanes 0..7 give the row addresses of the first matrix,
// lanes 8..15 those of the second (16-byte aligned); lane (g, t) receives elements [2t][g], [2t + 1][g] of each.
__device__ __forceinline__ void ldmatrix_x2_t(uint32_t& r0, uint32_t& r1, uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}

// term 0, 1, 2 of v = hi + mid + lo (bf16 each), as bit patterns
__device__ __forceinline__ uint32_t bf16_term(float v, int term) {
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    const float r1 = v - __bfloat162float(hi);
    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
    const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
    const __nv_bfloat16 pick = term == 0 ? hi : (term == 1 ? mid : lo);
    return (uint32_t)__bfloat16_as_ushort(pick);
}

template <int KS>
__global__ void __launch_bounds__(kCmThreads, 5) conv_pool_mma_kernel(ConvMmaParams p) {
    extern __shared__ __align__(16) uint16_t img_s[];      // [k shifted copies][c_in][hp][wp] bf16 bit patterns, zero border
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;                  // fragment coordinates of this lane
    const int H = (p.ksize - 1) / 2;
    {
        const int vecs = p.ksize * p.copy / 8;              // whole 16-byte vectors: every size is a multiple of 8 elements
        for (int j = tid; j < vecs; j += kCmThreads) reinterpret_cast<uint4*>(img_s)[j] = make_uint4(0u, 0u, 0u, 0u);
    }
    // left operand: channels g and g + 8, taps k0, k0 + 1 and k0 + 8, k0 + 9, four registers per k-step and bf16 term
    uint32_t aw[KS][3][4];
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
        float wv[4][2];
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int ch = g + (q & 1) * 8, k = ks * 16 + 2 * t + (q >> 1) * 8 + e;
                wv[q][e] = (ch < p.c_out && k < p.taps) ? __ldg(p.weight + ch * p.taps + k) : 0.0f;
            }
#pragma unroll
        for (int tr = 0; tr < 3; ++tr)
#pragma unroll
            for (int q = 0; q < 4; ++q) aw[ks][tr][q] = bf16_term(wv[q][0], tr) | (bf16_term(wv[q][1], tr) << 16);
    }
    // Row address (bytes, relative to the pixels' own position) that this lane hands to ldmatrix in every k-step: lanes
    // 0..15 stand for taps 16 ks + lane.  Tap (ci, dy, dx) of the pixels at (y, x0 ..) is copy dx, plane ci, row y + dy,
    // column x0.  Rows past the last tap multiply zero taps; they repeat the first row of their 8-row matrix (the same
    // address: no extra shared-memory traffic).
    uint32_t tap_off[KS];
    const int kk = p.ksize * p.ksize;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
        int k = ks * 16 + (lane & 15);
        if (k >= p.taps) k &= ~7;
        if (k >= p.taps) k = 0;
        const int ci = k / kk, r = k - ci * kk, dy = r / p.ksize, dx = r - dy * p.ksize;
        tap_off[ks] = 2u * (uint32_t)(dx * p.copy + ci * p.plane + dy * p.wp);
    }
    const float b_lo = (p.bias && g < p.c_out) ? __ldg(p.bias + g) : 0.0f;
    const float b_hi = (p.bias && g + 8 < p.c_out) ? __ldg(p.bias + g + 8) : 0.0f;
    const float nb_lo = -b_lo, nb_hi = -b_hi;

    const int strips = p.width >> 4;
    const int ph = p.height / p.pool, pw = p.width / p.pool;
    const int units = strips * ph;
    const float inv_window = 1.0f / (float)(p.pool * p.pool);
    const int pool_shift = 31 - __clz(p.pool);              // the pooling side is a power of two
    const uint32_t img_base = smem_u32(img_s);

    auto place = [&](int v, const uint4& q) {
        // vector v = 8 adjacent pixels of one image row (the width is a multiple of 16); it goes into every shifted copy
        uint32_t ci, r, y, xx;
        p.by_pixels.divmod((uint32_t)(v * 8), ci, r);
        p.by_width.divmod(r, y, xx);
        uint16_t* home = img_s + (int)ci * p.plane + ((int)y + H) * p.wp + (int)xx + H;
        for (int d = 0; d < p.ksize; ++d) {
            uint16_t* dst = home + d * p.copy - d;
            const int shift = H - d;                        // element offset of dst from a 16-byte boundary
            if (shift == 0) {
                *reinterpret_cast<uint4*>(dst) = q;
            } else if (shift & 1) {
                dst[0] = (uint16_t)(q.x & 0xFFFFu);
                uint32_t* d32 = reinterpret_cast<uint32_t*>(dst + 1);
                d32[0] = (q.x >> 16) | (q.y << 16);
                d32[1] = (q.y >> 16) | (q.z << 16);
                d32[2] = (q.z >> 16) | (q.w << 16);
                dst[7] = (uint16_t)(q.w >> 16);
            } else {
                uint32_t* d32 = reinterpret_cast<uint32_t*>(dst);
                d32[0] = q.x; d32[1] = q.y; d32[2] = q.z; d32[3] = q.w;
            }
        }
    };

    for (int64_t img = blockIdx.x; img < p.n; img += gridDim.x) {
        __syncthreads();      // the previous image's readers are done; the first time: the border is zero
        {
            const uint4* row = reinterpret_cast<const uint4*>(p.x + img * p.row_stride);
            for (int v = tid; v < p.n_vec; v += kCmThreads) place(v, __ldg(row + v));
        }
        __syncthreads();
        float* out = p.phi + img * p.phi_stride;
        for (int unit = warp; unit < units; unit += kCmWarps) {
            uint32_t py, sx;
            p.by_strips.divmod((uint32_t)unit, py, sx);
            const int x0 = (int)sx << 4;
            float vacc[2][4];
#pragma unroll
            for (int tile = 0; tile < 2; ++tile)
#pragma unroll
                for (int e = 0; e < 4; ++e) vacc[tile][e] = 0.0f;
            for (int yy = 0; yy < p.pool; ++yy) {
                const uint32_t at = img_base + 2u * (uint32_t)(((int)py * p.pool + yy) * p.wp + x0);   // pixels x0 .. x0 + 7; + 16 bytes: the next 8
                uint32_t b[2][KS][2];
#pragma unroll
                for (int tile = 0; tile < 2; ++tile)
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) ldmatrix_x2_t(b[tile][ks][0], b[tile][ks][1], at + 16u * tile + tap_off[ks]);
                // the two pixel tiles' accumulators alternate, so that consecutive products do not wait for one another
                float c[2][4];
#pragma unroll
                for (int ks = 0; ks < KS; ++ks)
#pragma unroll
                    for (int tr = 0; tr < 3; ++tr)
#pragma unroll
                        for (int tile = 0; tile < 2; ++tile) {
                            if (ks == 0 && tr == 0) mma_bf16_16816_first(c[tile], aw[ks][tr], b[tile][ks][0], b[tile][ks][1]);
                            else mma_bf16_16816(c[tile], aw[ks][tr], b[tile][ks][0], b[tile][ks][1]);
                        }
                // rectifier and the vertical part of the window.  The accumulators hold a - bias: max(a, 0) = max(a - bias, -bias)
                // + bias, and the bias goes in once per window below.
#pragma unroll
                for (int tile = 0; tile < 2; ++tile) {
                    vacc[tile][0] += fmaxf(c[tile][0], nb_lo);
                    vacc[tile][1] += fmaxf(c[tile][1], nb_lo);
                    vacc[tile][2] += fmaxf(c[tile][2], nb_hi);
                    vacc[tile][3] += fmaxf(c[tile][3], nb_hi);
                }
            }
            {
                // every entry has added up `pool` rows
                const float rows = (float)p.pool;
#pragma unroll
                for (int tile = 0; tile < 2; ++tile) {
                    vacc[tile][0] = fmaf(rows, b_lo, vacc[tile][0]);
                    vacc[tile][1] = fmaf(rows, b_lo, vacc[tile][1]);
                    vacc[tile][2] = fmaf(rows, b_hi, vacc[tile][2]);
                    vacc[tile][3] = fmaf(rows, b_hi, vacc[tile][3]);
                }
            }
            // The horizontal part.  Entries 0, 1 of a fragment: channel g, pixels 2t, 2t + 1 of the tile; entries 2, 3:
            // channel g + 8, the same pixels.
            if (p.pool == 1) {
#pragma unroll
                for (int tile = 0; tile < 2; ++tile)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int ch = g + (e >> 1) * 8, px = x0 + tile * 8 + 2 * t + (e & 1);
                        if (ch < p.c_out) out[(ch * ph + (int)py) * pw + px] = vacc[tile][e];
                    }
            } else {
                float s_lo[2], s_hi[2];
#pragma unroll
                for (int tile = 0; tile < 2; ++tile) {
                    s_lo[tile] = vacc[tile][0] + vacc[tile][1];
                    s_hi[tile] = vacc[tile][2] + vacc[tile][3];
                    if (p.pool >= 4) {
                        s_lo[tile] += __shfl_xor_sync(0xFFFFFFFFu, s_lo[tile], 1);
                        s_hi[tile] += __shfl_xor_sync(0xFFFFFFFFu, s_hi[tile], 1);
                    }
                    if (p.pool >= 8) {
                        s_lo[tile] += __shfl_xor_sync(0xFFFFFFFFu, s_lo[tile], 2);
                        s_hi[tile] += __shfl_xor_sync(0xFFFFFFFFu, s_hi[tile], 2);
                    }
                }
                if (p.pool == 16) {
                    s_lo[0] += s_lo[1];
                    s_hi[0] += s_hi[1];
                }
                const bool writer = p.pool == 2 || (p.pool == 4 && (t & 1) == 0) || (p.pool >= 8 && t == 0);
                if (writer) {
#pragma unroll
                    for (int tile = 0; tile < 2; ++tile) {
                        if (tile == 1 && p.pool == 16) break;
                        const int px = (x0 + tile * 8 + 2 * t) >> pool_shift;
                        float* o = out + (int)py * pw + px;
                        if (g < p.c_out) o[g * ph * pw] = s_lo[tile] * inv_window;
                        if (g + 8 < p.c_out) o[(g + 8) * ph * pw] = s_hi[tile] * inv_window;
                    }
                }
            }
        }
    }
}

// How many of the 8 row reads of each ldmatrix phase fall into the same 16-byte column of shared memory (0 = none):
// the eight rows of a matrix are eight taps, i.e. eight addresses that differ by copy, plane and row offsets.
int gather_conflicts(int c_in, int ksize, int wp, int plane, int copy) {
    const int taps = c_in * ksize * ksize, kk = ksize * ksize;
    int extra = 0;
    for (int m = 0; m * 8 < ((taps + 15) / 16) * 16; ++m) {
        int seen[8], n_seen = 0, used[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        for (int r = 0; r < 8; ++r) {
            int k = m * 8 + r;
            if (k >= taps) k &= ~7;
            if (k >= taps) k = 0;
            const int ci = k / kk, q = k - ci * kk, dy = q / ksize, dx = q - dy * ksize;
            const int vec = (dx * copy + ci * plane + dy * wp) / 8;          // 16-byte vector index
            bool dup = false;
            for (int s = 0; s < n_seen; ++s) dup |= seen[s] == vec;
            if (dup) continue;                                                // the same address: one read
            seen[n_seen++] = vec;
            extra += used[vec & 7];
            used[vec & 7] += 1;
        }
    }
    return extra;
}

// Row pitch, plane size and copy size with the fewest bank conflicts (a small search, remembered for the last shape).
void choose_layout(int c_in, int ksize, int width, int hp, int* wp_out, int* plane_out, int* copy_out) {
    static std::mutex mu;
    static int key[4] = {0, 0, 0, 0}, val[3] = {0, 0, 0};
    std::lock_guard<std::mutex> lock(mu);
    if (key[0] != c_in || key[1] != ksize || key[2] != width || key[3] != hp) {
        long best = -1;
        const int wp0 = (width + ksize - 1 + 7) / 8 * 8;
        for (int wp = wp0; wp <= wp0 + 56; wp += 8)
            for (int pe = 0; pe <= 56; pe += 8)
                for (int ce = 0; ce <= 56; ce += 8) {
                    const int plane = hp * wp + pe, copy = c_in * plane + ce;
                    const long cost = (long)gather_conflicts(c_in, ksize, wp, plane, copy) * 1000000 + (long)ksize * copy;   // ties: the smaller image
                    if (best < 0 || cost < best) best = cost, val[0] = wp, val[1] = plane, val[2] = copy;
                }
        key[0] = c_in; key[1] = ksize; key[2] = width; key[3] = hp;
    }
    *wp_out = val[0];
    *plane_out = val[1];
    *copy_out = val[2];
}

}  // namespace

// AA_ERR_UNSUPPORTED when the shape is not one this kernel covers (the caller then takes the multiply-add kernel).
aa_status launch_conv_pool_features_mma(aa_ctx_impl* c, const void* x, int dtype, int64_t n, int64_t row_stride, const aa_conv& cv,
                                        float* phi, int64_t phi_stride) {
    const int taps = cv.c_in * cv.ksize * cv.ksize;
    if (dtype != AA_BF16 || (cv.ksize != 1 && cv.ksize != 3 && cv.ksize != 5) || taps > kCmMaxTaps || cv.c_out > kCmMaxChan) return AA_ERR_UNSUPPORTED;
    if (cv.width % 16 || (cv.pool != 1 && cv.pool != 2 && cv.pool != 4 && cv.pool != 8 && cv.pool != 16) || cv.height % cv.pool)
        return AA_ERR_UNSUPPORTED;
    if ((uintptr_t)x % 16 || (row_stride * 2) % 16) return AA_ERR_UNSUPPORTED;
    ConvMmaParams p;
    p.x = static_cast<const uint16_t*>(x);
    p.n = n;
    p.row_stride = row_stride;
    p.c_in = cv.c_in;
    p.height = cv.height;
    p.width = cv.width;
    p.c_out = cv.c_out;
    p.ksize = cv.ksize;
    p.pool = cv.pool;
    p.weight = cv.weight;
    p.bias = cv.bias;
    p.phi = phi;
    p.phi_stride = phi_stride;
    p.hp = cv.height + cv.ksize - 1;
    choose_layout(cv.c_in, cv.ksize, cv.width, p.hp, &p.wp, &p.plane, &p.copy);
    p.taps = taps;
    p.n_vec = cv.c_in * cv.height * cv.width / 8;
    const size_t smem = (size_t)cv.ksize * p.copy * sizeof(uint16_t);
    if (smem > 96 * 1024) return AA_ERR_UNSUPPORTED;
    p.by_pixels.set((uint32_t)(cv.height * cv.width));
    p.by_width.set((uint32_t)cv.width);
    p.by_strips.set((uint32_t)(cv.width / 16));
    const void* kernel = taps > 16 ? (const void*)conv_pool_mma_kernel<2> : (const void*)conv_pool_mma_kernel<1>;
    if (smem > 48 * 1024 && cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return AA_ERR_CUDA;
    int grid = resident_ctas(c, kernel, kCmThreads, smem);
    if (grid <= 0) return AA_ERR_CUDA;
    if (grid > n) grid = (int)n;
    void* args[] = {&p};
    if (cudaLaunchKernel(kernel, dim3(grid), dim3(kCmThreads), args, smem, c->stream) != cudaSuccess) return AA_ERR_CUDA;
    ++c->launches;
    return AA_OK;
}

}  // namespace aa
