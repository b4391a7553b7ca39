// Features of the convolutional Assistant for bf16 images, on the matrix instructions
// (Sec. "Learning to generate smart training batches", closing paragraph: convolution shared with the Boss -> pooling ->
// single linear layer; this kernel is the convolution, the rectifier and the average pooling).
//
// Per image the convolution is a small dense contraction: [pixels x taps] * [taps x channels] with taps = c_in * k * k
// (27 for a 3 x 3 window over 3 planes) and 16 channels.  A warp takes 16 adjacent pixels of an image row at a time:
//   left operand  (16 pixels x 16 taps, bf16): gathered from the image in shared memory, two taps per register
//   right operand (16 taps x 8 channels): the taps, fp32 split into three bf16 terms hi + mid + lo (exact: 3 x 8
//                 significant bits), held in registers for the whole kernel; the three products go into one accumulator
//   mma.sync.m16n8k16, fp32 accumulation: bf16 x bf16 products are exact in fp32, so the arithmetic is that of an fp32
//   multiply-add loop up to summation order.
// The rectifier and the pooling work on the accumulator fragments: a fragment row is a pixel, so the vertical part of a
// window is a running sum over the image rows a warp walks through and the horizontal part a few lane shuffles at the end.
//
// This is the library's only use of matrix instructions on a small contraction (N = 16): the per-thread multiply-add
// kernel (conv_features.cu) issues 23.6 k warp instructions per 32 x 32 image, this one about a quarter of that.
// Shapes it does not cover (fp32 images, more than 32 taps or 16 channels, widths that are not a multiple of 16, pooling
// sides other than 1, 2, 4, 8, 16) stay with the other kernel.
#include <cuda_bf16.h>

#include <mutex>

#include "aa_internal.cuh"

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
    int wp, hp;              // padded row pitch (elements, even) and padded height of the image in shared memory
    int plane;               // elements per image plane in shared memory (even, >= hp * wp)
    int taps;
    int n_vec;               // 16-byte vectors per image
    FastDivM by_pixels, by_width, by_strips;
};

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// the same with the addend given apart from the result (the first product of an accumulator starts from the bias)
__device__ __forceinline__ void mma_bf16_16816_from(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1, float c_even, float c_odd) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%10, %11, %10, %11};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(c_even), "f"(c_odd));
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

template <int KS, int NT>
__global__ void __launch_bounds__(kCmThreads, 5) conv_pool_mma_kernel(ConvMmaParams p) {
    extern __shared__ __align__(16) uint16_t img_s[];      // [c_in][hp][wp] bf16 bit patterns, zero border
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;                  // fragment coordinates of this lane
    const int H = (p.ksize - 1) / 2;
    const int img_elems = p.c_in * p.plane;                 // even: the plane size is even
    for (int j = tid; j < img_elems / 2; j += kCmThreads) reinterpret_cast<uint32_t*>(img_s)[j] = 0u;

    // right operand: taps k0, k0 + 1 (and k0 + 8, k0 + 9) of channel nt * 8 + g, one register pair per bf16 term
    uint32_t bw[KS][NT][3][2];
    const int kk = p.ksize * p.ksize;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int ch = nt * 8 + g;
            float wv[4];
#pragma unroll
            for (int s = 0; s < 4; ++s) {
                const int k = ks * 16 + 2 * t + (s & 1) + (s >> 1) * 8;
                wv[s] = (ch < p.c_out && k < p.taps) ? __ldg(p.weight + ch * p.taps + k) : 0.0f;
            }
#pragma unroll
            for (int tr = 0; tr < 3; ++tr) {
                bw[ks][nt][tr][0] = bf16_term(wv[0], tr) | (bf16_term(wv[1], tr) << 16);
                bw[ks][nt][tr][1] = bf16_term(wv[2], tr) | (bf16_term(wv[3], tr) << 16);
            }
        }
    // where this lane's four operand slots of every k-step sit relative to a pixel: tap (ci, dy, dx) of pixel (y, x) is at
    // padded row y + dy, column x + dx.  Slots past the last tap multiply zero taps; they read an earlier tap (any in-window value does).
    int off[KS][4];
#pragma unroll
    for (int ks = 0; ks < KS; ++ks)
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            int k = ks * 16 + 2 * t + (s & 1) + (s >> 1) * 8;
            while (k >= p.taps && k >= 4) k -= 4;           // the tap a neighbouring lane reads: the same shared-memory words
            if (k >= p.taps) k = 0;
            const int ci = k / kk, r = k - ci * kk, dy = r / p.ksize, dx = r - dy * p.ksize;
            off[ks][s] = ci * p.plane + dy * p.wp + dx;
        }
    float bv[NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int ch = nt * 8 + 2 * t + e;
            bv[nt][e] = (p.bias && ch < p.c_out) ? __ldg(p.bias + ch) : 0.0f;
        }

    const int strips = p.width >> 4;
    const int ph = p.height / p.pool, pw = p.width / p.pool;
    const int units = strips * ph;
    const float inv_window = 1.0f / (float)(p.pool * p.pool);
    const int pool_shift = 31 - __clz(p.pool);              // the pooling side is a power of two
    const int group = p.pool < 8 ? p.pool : 8;              // pixels of one fragment half that share a window

    constexpr int kPre = 1;                                 // vectors of the next image a thread holds during the computation
    const bool prefetch = p.n_vec <= kPre * kCmThreads;
    uint4 pre[kPre];
    auto fetch = [&](int64_t img) {
        const uint4* row = reinterpret_cast<const uint4*>(p.x + img * p.row_stride);
#pragma unroll
        for (int u = 0; u < kPre; ++u) {
            const int v = tid + u * kCmThreads;
            if (v < p.n_vec) pre[u] = __ldg(row + v);
        }
    };
    auto place = [&](int v, const uint4& q) {
        // vector v = 8 adjacent pixels of one image row (the width is a multiple of 16)
        uint32_t ci, r, y, xx;
        p.by_pixels.divmod((uint32_t)(v * 8), ci, r);
        p.by_width.divmod(r, y, xx);
        uint16_t* dst = img_s + (int)ci * p.plane + ((int)y + H) * p.wp + (int)xx + H;
        if (H & 1) {
            // odd element offset: one 16-bit store, three aligned 32-bit stores, one 16-bit store
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
    };
    if (prefetch && blockIdx.x < p.n) fetch(blockIdx.x);

    for (int64_t img = blockIdx.x; img < p.n; img += gridDim.x) {
        __syncthreads();      // the previous image's readers are done; the first time: the border is zero
        if (prefetch) {
#pragma unroll
            for (int u = 0; u < kPre; ++u) {
                const int v = tid + u * kCmThreads;
                if (v < p.n_vec) place(v, pre[u]);
            }
            if (img + gridDim.x < p.n) fetch(img + gridDim.x);
        } else {
            const uint4* row = reinterpret_cast<const uint4*>(p.x + img * p.row_stride);
            for (int v = tid; v < p.n_vec; v += kCmThreads) place(v, __ldg(row + v));
        }
        __syncthreads();
        float* out = p.phi + img * p.phi_stride;
        for (int unit = warp; unit < units; unit += kCmWarps) {
            uint32_t py, sx;
            p.by_strips.divmod((uint32_t)unit, py, sx);
            const int x0 = (int)sx << 4;
            float vacc[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) vacc[nt][e] = 0.0f;
            for (int yy = 0; yy < p.pool; ++yy) {
                const uint16_t* px0 = img_s + ((int)py * p.pool + yy) * p.wp + x0 + g;     // pixel x0 + g; + 8: pixel x0 + g + 8
                float c[NT][4];
                uint32_t a[KS][4];
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    a[ks][0] = (uint32_t)px0[off[ks][0]] | ((uint32_t)px0[off[ks][1]] << 16);
                    a[ks][1] = (uint32_t)px0[off[ks][0] + 8] | ((uint32_t)px0[off[ks][1] + 8] << 16);
                    a[ks][2] = (uint32_t)px0[off[ks][2]] | ((uint32_t)px0[off[ks][3]] << 16);
                    a[ks][3] = (uint32_t)px0[off[ks][2] + 8] | ((uint32_t)px0[off[ks][3] + 8] << 16);
                }
                // the channel tiles' accumulators alternate, so that consecutive products do not wait for one another
#pragma unroll
                for (int ks = 0; ks < KS; ++ks)
#pragma unroll
                    for (int tr = 0; tr < 3; ++tr)
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            if (ks == 0 && tr == 0) mma_bf16_16816_from(c[nt], a[ks], bw[ks][nt][tr][0], bw[ks][nt][tr][1], bv[nt][0], bv[nt][1]);
                            else mma_bf16_16816(c[nt], a[ks], bw[ks][nt][tr][0], bw[ks][nt][tr][1]);
                        }
                // rectifier and the vertical part of the window (fragment rows are pixels of one image row)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) vacc[nt][e] += fmaxf(c[nt][e], 0.0f);
            }
            // the horizontal part: fragment rows g (entries 0, 1) and g + 8 (entries 2, 3) are adjacent pixels, lanes 4 apart
            // hold adjacent fragment rows
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                if (p.pool == 16) {
                    vacc[nt][0] += vacc[nt][2];
                    vacc[nt][1] += vacc[nt][3];
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (p.pool >= 2) vacc[nt][e] += __shfl_xor_sync(0xFFFFFFFFu, vacc[nt][e], 4);
                    if (p.pool >= 4) vacc[nt][e] += __shfl_xor_sync(0xFFFFFFFFu, vacc[nt][e], 8);
                    if (p.pool >= 8) vacc[nt][e] += __shfl_xor_sync(0xFFFFFFFFu, vacc[nt][e], 16);
                }
            }
            if ((g & (group - 1)) == 0) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int ch = nt * 8 + 2 * t + (e & 1);
                        if (ch < p.c_out && (p.pool < 16 || e < 2)) {
                            const int px = (x0 + g + ((e >> 1) << 3)) >> pool_shift;
                            out[(ch * ph + (int)py) * pw + px] = vacc[nt][e] * inv_window;
                        }
                    }
            }
        }
    }
}

}  // namespace

// Shared-memory wavefronts per operand load (1 = conflict-free) for a row pitch and plane size: the four lanes that share
// a fragment row read four different taps, eight adjacent pixels each.
static double gather_wavefronts(int c_in, int ksize, int wp, int plane) {
    const int taps = c_in * ksize * ksize, kk = ksize * ksize, k_steps = taps > 16 ? 2 : 1;
    int total = 0, count = 0;
    for (int ks = 0; ks < k_steps; ++ks)
        for (int s = 0; s < 4; ++s)
            for (int half = 0; half < 16; half += 8) {
                int words[32][8], n_words[32];               // distinct 32-bit words per bank
                for (int b = 0; b < 32; ++b) n_words[b] = 0;
                int worst = 1;
                for (int t = 0; t < 4; ++t) {
                    int k = ks * 16 + 2 * t + (s & 1) + (s >> 1) * 8;
                    while (k >= taps && k >= 4) k -= 4;
                    if (k >= taps) k = 0;
                    const int ci = k / kk, r = k - ci * kk, dy = r / ksize, dx = r - dy * ksize;
                    for (int g = 0; g < 8; ++g) {
                        const int word = (ci * plane + dy * wp + dx + g + half) >> 1, bank = word & 31;
                        bool seen = false;
                        for (int q = 0; q < n_words[bank]; ++q) seen |= words[bank][q] == word;
                        if (!seen && n_words[bank] < 8) words[bank][n_words[bank]++] = word;
                        if (n_words[bank] > worst) worst = n_words[bank];
                    }
                }
                total += worst;
                ++count;
            }
    return (double)total / count;
}

// Row pitch and plane size with the fewest bank conflicts for the gathers (a small search, remembered for the last shape).
static void choose_layout(int c_in, int ksize, int width, int hp, int* wp_out, int* plane_out) {
    static std::mutex mu;
    static int key[4] = {0, 0, 0, 0}, val[2] = {0, 0};
    std::lock_guard<std::mutex> lock(mu);
    if (key[0] == c_in && key[1] == ksize && key[2] == width && key[3] == hp) {
        *wp_out = val[0];
        *plane_out = val[1];
        return;
    }
    double best = 1e30;
    for (int wp = width + 4; wp <= width + 20; wp += 2)
        for (int extra = 0; extra <= 30; extra += 2) {
            const int plane = hp * wp + extra;
            const double w = gather_wavefronts(c_in, ksize, wp, plane) + 1e-6 * (double)plane;   // ties: the smaller image
            if (w < best) best = w, val[0] = wp, val[1] = plane;
        }
    key[0] = c_in; key[1] = ksize; key[2] = width; key[3] = hp;
    *wp_out = val[0];
    *plane_out = val[1];
}

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
    choose_layout(cv.c_in, cv.ksize, cv.width, p.hp, &p.wp, &p.plane);   // wp >= width + 4 (border of a 5 x 5 window), both even
    p.taps = taps;
    p.n_vec = cv.c_in * cv.height * cv.width / 8;
    const size_t smem = (size_t)cv.c_in * p.plane * sizeof(uint16_t);
    if (smem > 96 * 1024) return AA_ERR_UNSUPPORTED;
    p.by_pixels.set((uint32_t)(cv.height * cv.width));
    p.by_width.set((uint32_t)cv.width);
    p.by_strips.set((uint32_t)(cv.width / 16));
    const bool two_k = taps > 16, two_n = cv.c_out > 8;
    const void* kernel = two_k ? (two_n ? (const void*)conv_pool_mma_kernel<2, 2> : (const void*)conv_pool_mma_kernel<2, 1>)
                               : (two_n ? (const void*)conv_pool_mma_kernel<1, 2> : (const void*)conv_pool_mma_kernel<1, 1>);
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
