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
// zero border) and the taps in shared memory; a thread computes 8 adjacent outputs of four channels at a time, so that
// every value read from shared memory feeds about four multiply-adds; the rectified outputs meet in shared memory and
// are averaged window by window in a fixed order.
#include "aa_internal.cuh"

namespace aa {

namespace {

constexpr int kConvThreads = 256;
constexpr int kSeg = 8;                 // adjacent outputs per thread and pass
constexpr int kChan = 4;                // output channels per thread and pass

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
};

template <typename T, int K>
__global__ void __launch_bounds__(kConvThreads) conv_pool_features_kernel(ConvParams p) {
    extern __shared__ __align__(16) float conv_smem[];
    constexpr int H = (K - 1) / 2;
    const int taps = p.c_in * K * K;
    float* w_s = conv_smem;                                  // [c_out][c_in][K][K]
    float* b_s = w_s + p.c_out * taps;                       // [c_out]
    float* img_s = b_s + ((p.c_out + 3) & ~3);               // [c_in][hp][wp], zero border
    float* act_s = img_s + p.c_in * p.hp * p.wp;             // [c_out][height][act_pitch] rectified outputs, hpool of them per entry
    const int tid = threadIdx.x;
    for (int j = tid; j < p.c_out * taps; j += kConvThreads) w_s[j] = p.weight[j];
    for (int j = tid; j < p.c_out; j += kConvThreads) b_s[j] = p.bias ? p.bias[j] : 0.0f;
    for (int j = tid; j < p.c_in * p.hp * p.wp; j += kConvThreads) img_s[j] = 0.0f;

    const int segs = (p.width + kSeg - 1) / kSeg;
    const int quads = (p.c_out + kChan - 1) / kChan;
    const int items = quads * p.height * segs;
    const int pixels = p.height * p.width;
    const int ph = p.height / p.pool, pw = p.width / p.pool;
    const int feats = p.c_out * ph * pw;
    const float inv_window = 1.0f / (float)(p.pool * p.pool);
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
                    const int j = v * VE;
                    const int ci = j / pixels, r = j - ci * pixels;
                    const int y = r / p.width, xx = r - y * p.width;
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
            const int seg = item % segs;
            const int y = (item / segs) % p.height;
            const int cq = item / (segs * p.height);
            int co[kChan];
            float acc[kChan][kSeg];
#pragma unroll
            for (int c = 0; c < kChan; ++c) {
                co[c] = cq * kChan + c < p.c_out ? cq * kChan + c : p.c_out - 1;     // a short last group repeats its last channel
#pragma unroll
                for (int q = 0; q < kSeg; ++q) acc[c][q] = b_s[co[c]];
            }
            for (int ci = 0; ci < p.c_in; ++ci) {
#pragma unroll
                for (int dy = 0; dy < K; ++dy) {
                    const float* in_row = img_s + (ci * p.hp + y + dy) * p.wp + seg * kSeg;
                    float in[kSeg + K - 1];
#pragma unroll
                    for (int q = 0; q < kSeg + K - 1; ++q) in[q] = in_row[q];
#pragma unroll
                    for (int dx = 0; dx < K; ++dx) {
#pragma unroll
                        for (int c = 0; c < kChan; ++c) {
                            const float t = w_s[co[c] * taps + (ci * K + dy) * K + dx];
#pragma unroll
                            for (int q = 0; q < kSeg; ++q) acc[c][q] = fmaf(t, in[q + dx], acc[c][q]);
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
            const int px = f % pw, py = (f / pw) % ph, co = f / (pw * ph);
            const int across = p.pool / p.hpool;          // partial sums per window row
            const float* a = act_s + (co * p.height + py * p.pool) * p.act_pitch + px * across;
            float sum = 0.0f;
            for (int yy = 0; yy < p.pool; ++yy)
                for (int xx = 0; xx < across; ++xx) sum += a[yy * p.act_pitch + xx];
            out[f] = sum * inv_window;
        }
    }
}

}  // namespace

aa_status launch_conv_pool_features(aa_ctx_impl* c, const void* x, int dtype, int64_t n, int64_t row_stride, const aa_conv& cv,
                                    float* phi, int64_t phi_stride) {
    if (cv.ksize != 1 && cv.ksize != 3 && cv.ksize != 5) return AA_ERR_UNSUPPORTED;
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
    p.wp = segs * kSeg + cv.ksize - 1;
    if ((p.wp & 1) == 0) ++p.wp;          // odd pitch: rows of adjacent segments fall into different banks
    p.hp = cv.height + cv.ksize - 1;
    const int es = dtype == AA_BF16 ? 2 : 4;
    p.vec_rows = ((uintptr_t)x % 16 == 0 && (row_stride * es) % 16 == 0 && cv.width % (16 / es) == 0) ? 1 : 0;
    p.hpool = (cv.pool == 2 || cv.pool == 4 || cv.pool == 8) ? cv.pool : ((cv.pool % 8 == 0) ? 8 : 1);
    if (cv.width % p.hpool) p.hpool = 1;
    p.act_pitch = ((segs * kSeg) / p.hpool) | 1;
    const size_t floats = (size_t)cv.c_out * cv.c_in * cv.ksize * cv.ksize + ((cv.c_out + 3) & ~3) + (size_t)cv.c_in * p.hp * p.wp +
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
