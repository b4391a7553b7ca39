// Features of the convolutional Assistant (Sec. "Learning to generate smart training batches", closing paragraph: for
// image tasks the Assistant may be a convolution layer sharing its parameters with the Boss, then a pooling layer, then
// a single linear layer).  This kernel is the first two layers: per instance (an image stored channel-major)
//   a[co][y][x]   = bias[co] + sum_{ci, dy, dx} weight[co][ci][dy][dx] * image[ci][y + dy - h][x + dx - h]     (zero padding)
//   phi[co][py][px] = mean over the pool x pool window of max(a, 0)
// in fp32.  The single linear layer on phi is the library's linear Assistant (scoring, shrinking, update), so only
// phi is computed here; the convolution weights are the Boss's and are not trained by the Assistant.
//
// The work is plain fp32 arithmetic (27 multiply-adds per output value for a 3 x 3 x 3 window, 0.44 M per 32 x 32 image
// with 16 channels) against 6 KB of input per image: ALU-bound, not memory-bound.  One CTA holds an image (with its
// zero border) and the taps in shared memory; a thread computes 8 adjacent outputs of four channels at a time and reads
// shared memory in 16-byte vectors only (three of the image row and one of taps per filter position feed 96 multiply-adds);
// the rectified outputs meet in shared memory and are averaged window by window in a fixed order.
#include "aa_internal.cuh"

namespace aa {

namespace {

constexpr int kConvThreads = 256;
constexpr int kSeg = 8;                 // adjacent outputs per thread and pass
constexpr int kChan = 4;                // output channels per thread and pass

// Division of a small index by a divisor fixed per launch: one multiply-high instead of the integer-division sequence.
// magic = floor(2^32 / d) + 1 gives the exact quotient whenever n * d < 2^32; every index here is below the number of
// floats of an image in shared memory (< 2^16) and so is every divisor.  d = 1 is encoded as magic 0.
struct FastDiv {
    uint32_t d, magic;
    __host__ void set(uint32_t divisor) {
        d = divisor;
        magic = divisor <= 1 ? 0u : (uint32_t)((1ull << 32) / divisor + 1ull);
    }
    __device__ __forceinline__ uint32_t div(uint32_t n) const { return magic ? __umulhi(n, magic) : n; }
    __device__ __forceinline__ void divmod(uint32_t n, uint32_t& q, uint32_t& r) const {
        q = div(n);
        r = n - q * d;
    }
};

struct ConvParams {
    const void* x;
    int64_t n, row_stride;
    int c_in, height, width, c_out, pool;
    const float* weight;
    const float* bias;
    float* phi;
    int64_t phi_stride;
    int wp;        // padded row width in shared memory
    int hp;        // padded image height
    int vec_rows;  // image rows can be read with 16-byte loads
    int hpool;     // adjacent outputs a thread adds up before storing (1, 2, 4 or 8; divides pool)
    int act_pitch; // floats per row of the rectified (partly pooled) outputs in shared memory, odd
    FastDiv by_pixels, by_width, by_segs, by_height, by_pw, by_ph;
};

template <typename T, int K>
__global__ void __launch_bounds__(kConvThreads) conv_pool_features_kernel(ConvParams p) {
    extern __shared__ __align__(16) float conv_smem[];
    constexpr int H = (K - 1) / 2;
    const int taps = p.c_in * K * K;
    const int segs = (p.width + kSeg - 1) / kSeg;
    const int quads = (p.c_out + kChan - 1) / kChan;
    float* w_s = conv_smem;                                  // [quads][c_in][K][K][4]: the four channels of a group side by side
    float* b_s = w_s + quads * taps * kChan;                 // [quads][4]; channels past c_out have zero taps and bias
    float* img_s = b_s + quads * kChan;                      // [c_in][hp][wp], zero border, rows 16-byte aligned
    float* act_s = img_s + p.c_in * p.hp * p.wp;             // [c_out][height][act_pitch] rectified outputs, hpool of them per entry
    const int tid = threadIdx.x;
    for (int j = tid; j < quads * taps * kChan; j += kConvThreads) {
        const int c = j % kChan, t = (j / kChan) % taps, co = (j / (kChan * taps)) * kChan + c;
        w_s[j] = co < p.c_out ? p.weight[co * taps + t] : 0.0f;
    }
    for (int j = tid; j < quads * kChan; j += kConvThreads) b_s[j] = (p.bias && j < p.c_out) ? p.bias[j] : 0.0f;
    for (int j = tid; j < p.c_in * p.hp * p.wp; j += kConvThreads) img_s[j] = 0.0f;

    const int items = quads * p.height * segs;
    const int pixels = p.height * p.width;
    const int ph = p.height / p.pool, pw = p.width / p.pool;
    const int feats = p.c_out * ph * pw;
    const float inv_window = 1.0f / (float)(p.pool * p.pool);
    const int across = p.pool / p.hpool;               // partial sums per window row in act_s
    const T* base = static_cast<const T*>(p.x);

    constexpr int VE = Vec<T>::kElems;
    constexpr int kPre = 2;                        // vectors of the next image a thread holds while the current one is computed
    const int n_vec = p.c_in * pixels / VE;
    const bool prefetch = p.vec_rows && n_vec <= kPre * kConvThreads;
    uint4 pre[kPre];
    auto fetch = [&](int64_t img) {
        const T* row = base + img * p.row_stride;
#pragma unroll
        for (int u = 0; u < kPre; ++u) {
            const int v = tid + u * kConvThreads;
            if (v < n_vec) pre[u] = __ldg(reinterpret_cast<const uint4*>(row) + v);
        }
    };
    if (prefetch && blockIdx.x < p.n) fetch(blockIdx.x);

    for (int64_t img = blockIdx.x; img < p.n; img += gridDim.x) {
        __syncthreads();      // the previous image's readers are done; the first time: taps and border are in place
        const T* row = base + img * p.row_stride;
        if (prefetch) {
            // this image's vectors were requested while the previous image was computed (a vector never straddles an
            // image row: the width is a whole number of vectors)
#pragma unroll
            for (int u = 0; u < kPre; ++u) {
                const int v = tid + u * kConvThreads;
                if (v < n_vec) {
                    uint32_t ci, r, y, xx;
                    p.by_pixels.divmod((uint32_t)(v * VE), ci, r);
                    p.by_width.divmod(r, y, xx);
                    float e[VE];
                    Vec<T>::unpack(pre[u], e);
                    float* dst = img_s + (ci * p.hp + y + H) * p.wp + xx + H;
#pragma unroll
                    for (int q = 0; q < VE; ++q) dst[q] = e[q];
                }
            }
            if (img + gridDim.x < p.n) fetch(img + gridDim.x);
        } else if (p.vec_rows) {
            for (int v = tid; v < n_vec; v += kConvThreads) {
                const int j = v * VE;
                const int ci = j / pixels, r = j - ci * pixels;
                const int y = r / p.width, xx = r - y * p.width;
                float e[VE];
                Vec<T>::load(row + j, e);
                float* dst = img_s + (ci * p.hp + y + H) * p.wp + xx + H;
#pragma unroll
                for (int q = 0; q < VE; ++q) dst[q] = e[q];
            }
        } else {
            for (int j = tid; j < p.c_in * pixels; j += kConvThreads) {
                const int ci = j / pixels, r = j - ci * pixels;
                const int y = r / p.width, xx = r - y * p.width;
                img_s[(ci * p.hp + y + H) * p.wp + xx + H] = Vec<T>::one(row + j);
            }
        }
        __syncthreads();
        for (int item = tid; item < items; item += kConvThreads) {
            uint32_t rest, useg, ucq, uy;
            p.by_segs.divmod((uint32_t)item, rest, useg);
            p.by_height.divmod(rest, ucq, uy);
            const int seg = (int)useg, y = (int)uy, cq = (int)ucq;
            int co[kChan];
            float acc[kChan][kSeg];
            {
                const float4 b4 = *reinterpret_cast<const float4*>(b_s + cq * kChan);
                const float bv[kChan] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
                for (int c = 0; c < kChan; ++c) {
                    co[c] = cq * kChan + c;
#pragma unroll
                    for (int q = 0; q < kSeg; ++q) acc[c][q] = bv[c];
                }
            }
            // 16-byte shared-memory reads only: kInVec vectors of the padded image row, one vector of taps per (ci, dy, dx)
            constexpr int kInVec = (kSeg + K - 1 + 3) / 4;
            const float4* tap = reinterpret_cast<const float4*>(w_s) + cq * taps;
            for (int ci = 0; ci < p.c_in; ++ci) {
#pragma unroll
                for (int dy = 0; dy < K; ++dy) {
                    const float4* in_row = reinterpret_cast<const float4*>(img_s + (ci * p.hp + y + dy) * p.wp + seg * kSeg);
                    float in[4 * kInVec];
#pragma unroll
                    for (int v = 0; v < kInVec; ++v) {
                        const float4 t = in_row[v];
                        in[4 * v] = t.x; in[4 * v + 1] = t.y; in[4 * v + 2] = t.z; in[4 * v + 3] = t.w;
                    }
#pragma unroll
                    for (int dx = 0; dx < K; ++dx) {
                        const float4 t4 = tap[(ci * K + dy) * K + dx];
                        const float tv[kChan] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
                        for (int c = 0; c < kChan; ++c) {
#pragma unroll
                            for (int q = 0; q < kSeg; ++q) acc[c][q] = fmaf(tv[c], in[q + dx], acc[c][q]);
                        }
                    }
                }
            }
            // rectifier, then the horizontal part of the pooling in registers (groups of hpool adjacent outputs, hpool = the
            // pooling side when it divides the 8 outputs of a thread, else 1): fewer, narrower stores
#pragma unroll
            for (int c = 0; c < kChan; ++c) {
                if (cq * kChan + c < p.c_out) {
                    float* dst = act_s + (co[c] * p.height + y) * p.act_pitch + (seg * kSeg) / p.hpool;
                    if (p.hpool == 4) {
                        const int x0 = seg * kSeg;
                        if (x0 < p.width) dst[0] = fmaxf(acc[c][0], 0.0f) + fmaxf(acc[c][1], 0.0f) + fmaxf(acc[c][2], 0.0f) + fmaxf(acc[c][3], 0.0f);
                        if (x0 + 4 < p.width) dst[1] = fmaxf(acc[c][4], 0.0f) + fmaxf(acc[c][5], 0.0f) + fmaxf(acc[c][6], 0.0f) + fmaxf(acc[c][7], 0.0f);
                    } else if (p.hpool == 8) {
                        float t = 0.0f;
#pragma unroll
                        for (int q = 0; q < kSeg; ++q) t += fmaxf(acc[c][q], 0.0f);
                        if (seg * kSeg < p.width) dst[0] = t;
                    } else if (p.hpool == 2) {
#pragma unroll
                        for (int q = 0; q < kSeg; q += 2)
                            if (seg * kSeg + q < p.width) dst[q >> 1] = fmaxf(acc[c][q], 0.0f) + fmaxf(acc[c][q + 1], 0.0f);
                    } else {
#pragma unroll
                        for (int q = 0; q < kSeg; ++q)
                            if (seg * kSeg + q < p.width) dst[q] = fmaxf(acc[c][q], 0.0f);
                    }
                }
            }
        }
        __syncthreads();
        float* out = p.phi + img * p.phi_stride;
        for (int f = tid; f < feats; f += kConvThreads) {
            uint32_t rest, px, co, py;
            p.by_pw.divmod((uint32_t)f, rest, px);
            p.by_ph.divmod(rest, co, py);
            const float* a = act_s + ((int)co * p.height + (int)py * p.pool) * p.act_pitch + (int)px * across;
            float sum = 0.0f;
            if (across == 1) {
                // the usual case (the pooling side divides a thread's 8 outputs): one partial sum per window row
#pragma unroll 4
                for (int yy = 0; yy < p.pool; ++yy) sum += a[yy * p.act_pitch];
            } else {
                for (int yy = 0; yy < p.pool; ++yy)
                    for (int xx = 0; xx < across; ++xx) sum += a[yy * p.act_pitch + xx];
            }
            out[f] = sum * inv_window;
        }
    }
}

}  // namespace

// bf16 images of the common shapes go to the matrix-instruction kernel (conv_features_mma.cu)
aa_status launch_conv_pool_features_mma(aa_ctx_impl* c, const void* x, int dtype, int64_t n, int64_t row_stride, const aa_conv& cv,
                                        float* phi, int64_t phi_stride);

aa_status launch_conv_pool_features(aa_ctx_impl* c, const void* x, int dtype, int64_t n, int64_t row_stride, const aa_conv& cv,
                                    float* phi, int64_t phi_stride) {
    if (cv.ksize != 1 && cv.ksize != 3 && cv.ksize != 5) return AA_ERR_UNSUPPORTED;
    {
        const aa_status st = launch_conv_pool_features_mma(c, x, dtype, n, row_stride, cv, phi, phi_stride);
        if (st != AA_ERR_UNSUPPORTED) return st;
    }
    ConvParams p;
    p.x = x;
    p.n = n;
    p.row_stride = row_stride;
    p.c_in = cv.c_in;
    p.height = cv.height;
    p.width = cv.width;
    p.c_out = cv.c_out;
    p.pool = cv.pool;
    p.weight = cv.weight;
    p.bias = cv.bias;
    p.phi = phi;
    p.phi_stride = phi_stride;
    const int segs = (cv.width + kSeg - 1) / kSeg;
    // rows of whole 16-byte vectors with one spare vector (the last segment reads up to 4 floats past its 8 outputs); with
    // a 32-wide image the pitch of 36 floats puts the eight vectors a quarter-warp reads into eight different bank groups
    p.wp = segs * kSeg + 4;
    p.hp = cv.height + cv.ksize - 1;
    const int es = dtype == AA_BF16 ? 2 : 4;
    p.vec_rows = ((uintptr_t)x % 16 == 0 && (row_stride * es) % 16 == 0 && cv.width % (16 / es) == 0) ? 1 : 0;
    p.hpool = (cv.pool == 2 || cv.pool == 4 || cv.pool == 8) ? cv.pool : ((cv.pool % 8 == 0) ? 8 : 1);
    if (cv.width % p.hpool) p.hpool = 1;
    p.act_pitch = ((segs * kSeg) / p.hpool) | 1;
    p.by_pixels.set((uint32_t)(cv.height * cv.width));
    p.by_width.set((uint32_t)cv.width);
    p.by_segs.set((uint32_t)segs);
    p.by_height.set((uint32_t)cv.height);
    p.by_pw.set((uint32_t)(cv.width / cv.pool));
    p.by_ph.set((uint32_t)(cv.height / cv.pool));
    const size_t quads = (size_t)(cv.c_out + kChan - 1) / kChan;
    const size_t floats = quads * kChan * ((size_t)cv.c_in * cv.ksize * cv.ksize + 1) + (size_t)cv.c_in * p.hp * p.wp +
                          (size_t)cv.c_out * cv.height * p.act_pitch;
    const size_t smem = floats * sizeof(float);
    if (smem > 200 * 1024) return AA_ERR_UNSUPPORTED;
    const void* kernel;
    if (dtype == AA_BF16)
        kernel = cv.ksize == 1 ? (const void*)conv_pool_features_kernel<uint16_t, 1>
                 : cv.ksize == 3 ? (const void*)conv_pool_features_kernel<uint16_t, 3> : (const void*)conv_pool_features_kernel<uint16_t, 5>;
    else
        kernel = cv.ksize == 1 ? (const void*)conv_pool_features_kernel<float, 1>
                 : cv.ksize == 3 ? (const void*)conv_pool_features_kernel<float, 3> : (const void*)conv_pool_features_kernel<float, 5>;
    if (smem > 48 * 1024 && cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return AA_ERR_CUDA;
    int grid = resident_ctas(c, kernel, kConvThreads, smem);
    if (grid <= 0) return AA_ERR_CUDA;
    if (grid > n) grid = (int)n;
    void* args[] = {&p};
    if (cudaLaunchKernel(kernel, dim3(grid), dim3(kConvThreads), args, smem, c->stream) != cudaSuccess) return AA_ERR_CUDA;
    ++c->launches;
    return AA_OK;
}

}  // namespace aa
