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
// zero border) and the taps in shared memory; a thread computes 8 adjacent outputs of two channels at a time, so that
// every value read from shared memory feeds about five multiply-adds; the rectified outputs meet in shared memory and
// are averaged window by window in a fixed order.
#include "aa_internal.cuh"

namespace aa {

namespace {

constexpr int kConvThreads = 512;
constexpr int kSeg = 8;                 // adjacent outputs per thread and pass

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
};

template <typename T, int K>
__global__ void __launch_bounds__(kConvThreads) conv_pool_features_kernel(ConvParams p) {
    extern __shared__ __align__(16) float conv_smem[];
    constexpr int H = (K - 1) / 2;
    const int taps = p.c_in * K * K;
    float* w_s = conv_smem;                                  // [c_out][c_in][K][K]
    float* b_s = w_s + p.c_out * taps;                       // [c_out]
    float* img_s = b_s + ((p.c_out + 3) & ~3);               // [c_in][hp][wp], zero border
    float* act_s = img_s + p.c_in * p.hp * p.wp;             // [c_out][height][width] rectified outputs
    const int tid = threadIdx.x;
    for (int j = tid; j < p.c_out * taps; j += kConvThreads) w_s[j] = p.weight[j];
    for (int j = tid; j < p.c_out; j += kConvThreads) b_s[j] = p.bias ? p.bias[j] : 0.0f;
    for (int j = tid; j < p.c_in * p.hp * p.wp; j += kConvThreads) img_s[j] = 0.0f;

    const int segs = (p.width + kSeg - 1) / kSeg;
    const int pairs = (p.c_out + 1) / 2;
    const int items = pairs * p.height * segs;
    const int pixels = p.height * p.width;
    const int ph = p.height / p.pool, pw = p.width / p.pool;
    const int feats = p.c_out * ph * pw;
    const float inv_window = 1.0f / (float)(p.pool * p.pool);
    const T* base = static_cast<const T*>(p.x);

    for (int64_t img = blockIdx.x; img < p.n; img += gridDim.x) {
        __syncthreads();      // the previous image's readers are done; the first time: taps and border are in place
        const T* row = base + img * p.row_stride;
        for (int j = tid; j < p.c_in * pixels; j += kConvThreads) {
            const int ci = j / pixels, r = j - ci * pixels;
            const int y = r / p.width, xx = r - y * p.width;
            img_s[(ci * p.hp + y + H) * p.wp + xx + H] = Vec<T>::one(row + j);
        }
        __syncthreads();
        for (int item = tid; item < items; item += kConvThreads) {
            const int seg = item % segs;
            const int y = (item / segs) % p.height;
            const int cp = item / (segs * p.height);
            const int co0 = 2 * cp, co1 = co0 + 1 < p.c_out ? co0 + 1 : co0;
            float acc0[kSeg], acc1[kSeg];
#pragma unroll
            for (int q = 0; q < kSeg; ++q) { acc0[q] = b_s[co0]; acc1[q] = b_s[co1]; }
            const float* w0 = w_s + co0 * taps;
            const float* w1 = w_s + co1 * taps;
            for (int ci = 0; ci < p.c_in; ++ci) {
#pragma unroll
                for (int dy = 0; dy < K; ++dy) {
                    const float* in_row = img_s + (ci * p.hp + y + dy) * p.wp + seg * kSeg;
                    float in[kSeg + K - 1];
#pragma unroll
                    for (int q = 0; q < kSeg + K - 1; ++q) in[q] = in_row[q];
#pragma unroll
                    for (int dx = 0; dx < K; ++dx) {
                        const float t0 = w0[(ci * K + dy) * K + dx], t1 = w1[(ci * K + dy) * K + dx];
#pragma unroll
                        for (int q = 0; q < kSeg; ++q) {
                            acc0[q] = fmaf(t0, in[q + dx], acc0[q]);
                            acc1[q] = fmaf(t1, in[q + dx], acc1[q]);
                        }
                    }
                }
            }
#pragma unroll
            for (int q = 0; q < kSeg; ++q) {
                const int xx = seg * kSeg + q;
                if (xx < p.width) {
                    act_s[(co0 * p.height + y) * p.width + xx] = fmaxf(acc0[q], 0.0f);
                    if (co1 != co0) act_s[(co1 * p.height + y) * p.width + xx] = fmaxf(acc1[q], 0.0f);
                }
            }
        }
        __syncthreads();
        float* out = p.phi + img * p.phi_stride;
        for (int f = tid; f < feats; f += kConvThreads) {
            const int px = f % pw, py = (f / pw) % ph, co = f / (pw * ph);
            const float* a = act_s + (co * p.height + py * p.pool) * p.width + px * p.pool;
            float sum = 0.0f;
            for (int yy = 0; yy < p.pool; ++yy)
                for (int xx = 0; xx < p.pool; ++xx) sum += a[yy * p.width + xx];
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
    const size_t floats = (size_t)cv.c_out * cv.c_in * cv.ksize * cv.ksize + ((cv.c_out + 3) & ~3) + (size_t)cv.c_in * p.hp * p.wp +
                          (size_t)cv.c_out * cv.height * cv.width;
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
