// First convolution of an image network: 3 x 3, a handful of input channels (the colour planes), 32 or 64
// output channels, no bias, no activation (a batch norm follows).  With three input channels the reduction is only
// 27 long: the implicit-GEMM kernels spend their time on the index arithmetic of a gather that has no vectors to
// fetch, and the tensor-core kernels do not take it (their operand rows must be multiples of 16 bytes).  Here the
// whole filter bank sits in shared memory as float, a thread owns one output pixel with all its output channels
// in registers (forward), and the weight gradient is a small outer product per pixel that a warp accumulates in
// registers over its share of the pixels.
#include <cuda_bf16.h>
#include <algorithm>
#include <cstdint>
#include "kernels.h"
#include "launch.cuh"

namespace ftp {
namespace {

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }

template <int COUT> __device__ __forceinline__ void store_row(float* p, const float (&a)[COUT]) {
#pragma unroll
    for (int c = 0; c < COUT; c += 4) *reinterpret_cast<float4*>(p + c) = make_float4(a[c], a[c + 1], a[c + 2], a[c + 3]);
}
template <int COUT> __device__ __forceinline__ void store_row(__nv_bfloat16* p, const float (&a)[COUT]) {
#pragma unroll
    for (int c = 0; c < COUT; c += 8) {
        unsigned u[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(a[c + 2 * i], a[c + 2 * i + 1]);
            u[i] = *reinterpret_cast<const unsigned*>(&h);
        }
        *reinterpret_cast<uint4*>(p + c) = make_uint4(u[0], u[1], u[2], u[3]);
    }
}

// y[n][ho][wo][:] = sum over the 3 x 3 x CIN window of x * w[r][s][ci][:].  grid: ceil(pixels / 128), block 128.
template <typename T, int CIN, int COUT>
__global__ void __launch_bounds__(128) stem_fwd_kernel(const T* __restrict__ x, const T* __restrict__ w, T* __restrict__ y, int N, int H, int W, int Ho,
                                                       int Wo, int stride) {
    __shared__ __align__(16) float ws[9 * CIN][COUT];
    grid_dep_sync();
    for (int i = threadIdx.x; i < 9 * CIN * COUT; i += 128) ws[i / COUT][i % COUT] = to_f(w[i]);
    __syncthreads();
    const long long p = (long long)blockIdx.x * 128 + threadIdx.x;
    if (p >= (long long)N * Ho * Wo) return;
    const int wo = (int)(p % Wo);
    const long long q = p / Wo;
    const int ho = (int)(q % Ho), n = (int)(q / Ho);
    float acc[COUT];
#pragma unroll
    for (int c = 0; c < COUT; ++c) acc[c] = 0.f;
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        const int hi = ho * stride - 1 + r;
        if (hi < 0 || hi >= H) continue;
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            const int wi = wo * stride - 1 + s;
            if (wi < 0 || wi >= W) continue;
            const T* px = x + ((long long)(n * H + hi) * W + wi) * CIN;
#pragma unroll
            for (int ci = 0; ci < CIN; ++ci) {
                const float v = to_f(px[ci]);
                const float* wr = ws[(r * 3 + s) * CIN + ci];
#pragma unroll
                for (int c = 0; c < COUT; c += 4) {
                    const float4 k = *reinterpret_cast<const float4*>(wr + c);
                    acc[c] = fmaf(v, k.x, acc[c]); acc[c + 1] = fmaf(v, k.y, acc[c + 1]);
                    acc[c + 2] = fmaf(v, k.z, acc[c + 2]); acc[c + 3] = fmaf(v, k.w, acc[c + 3]);
                }
            }
        }
    }
    store_row<COUT>(y + p * COUT, acc);
}

// Weight gradient dw[r][s][ci][c] = sum over output pixels of x(window) * dy[c].  A warp takes 32 pixels at a time:
// lane p gathers the 9 * CIN window values of pixel p into shared memory and the warp copies the 32 rows of dy;
// then lane (r, ct) -- 3 filter rows x 8 groups of COUT / 8 channels, 24 lanes -- adds the 3 * CIN x COUT / 8 outer
// products of the 32 pixels to its registers.  The warps of a block are added in warp order and every block leaves
// one partial [9 * CIN][COUT]; the fixed-order second pass adds the blocks.  grid: `blocks`, block 128.
template <typename T, int CIN, int COUT>
__global__ void __launch_bounds__(128) stem_wgrad_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ partial, int N, int H, int W,
                                                         int Ho, int Wo, int stride) {
    constexpr int K = 9 * CIN, KR = 3 * CIN, CT = COUT / 8, XS = K + 1;
    __shared__ float xs[4][32][XS];
    __shared__ __align__(16) float ds[4][32][COUT];
    grid_dep_sync();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = lane / 8, ct = lane % 8;                     // lanes 24..31 only help with the staging
    const long long M = (long long)N * Ho * Wo, chunks = (M + 31) / 32;
    float acc[KR][CT];
#pragma unroll
    for (int k = 0; k < KR; ++k)
#pragma unroll
        for (int c = 0; c < CT; ++c) acc[k][c] = 0.f;
    for (long long ch = (long long)blockIdx.x * 4 + warp; ch < chunks; ch += (long long)gridDim.x * 4) {
        const long long p = ch * 32 + lane;
        {   // window of pixel p (zeros outside the image and past the last pixel)
            const bool live = p < M;
            const int wo = live ? (int)(p % Wo) : 0;
            const long long q = live ? p / Wo : 0;
            const int ho = (int)(q % Ho), n = (int)(q / Ho);
#pragma unroll
            for (int rr = 0; rr < 3; ++rr)
#pragma unroll
                for (int s = 0; s < 3; ++s) {
                    const int hi = ho * stride - 1 + rr, wi = wo * stride - 1 + s;
                    const bool in = live && hi >= 0 && hi < H && wi >= 0 && wi < W;
                    const T* px = x + ((long long)(n * H + hi) * W + wi) * CIN;
#pragma unroll
                    for (int ci = 0; ci < CIN; ++ci) xs[warp][lane][(rr * 3 + s) * CIN + ci] = in ? to_f(px[ci]) : 0.f;
                }
        }
        {   // the 32 rows of dy are contiguous: lanes stride through them
            const long long base = ch * 32 * COUT, end = M * COUT;
#pragma unroll 4
            for (int i = lane; i < 32 * COUT; i += 32) ds[warp][i / COUT][i % COUT] = base + i < end ? to_f(dy[base + i]) : 0.f;
        }
        __syncwarp();
        if (lane < 24) {
#pragma unroll 4
            for (int pp = 0; pp < 32; ++pp) {
                float xv[KR], dv[CT];
#pragma unroll
                for (int k = 0; k < KR; ++k) xv[k] = xs[warp][pp][r * KR + k];
#pragma unroll
                for (int c = 0; c < CT; c += 4) {
                    const float4 d = *reinterpret_cast<const float4*>(&ds[warp][pp][ct * CT + c]);
                    dv[c] = d.x; dv[c + 1] = d.y; dv[c + 2] = d.z; dv[c + 3] = d.w;
                }
#pragma unroll
                for (int k = 0; k < KR; ++k)
#pragma unroll
                    for (int c = 0; c < CT; ++c) acc[k][c] = fmaf(xv[k], dv[c], acc[k][c]);
            }
        }
        __syncwarp();
    }
    // the four warps in warp order through shared memory (the dy staging area is free now)
    __syncthreads();
    float* red = &ds[0][0][0];                                  // [4][K][COUT] floats needed: 4 * 32 * COUT available, K <= 32
    static_assert(K <= 32, "the reduction buffer is the dy staging area");
    if (lane < 24)
#pragma unroll
        for (int k = 0; k < KR; ++k)
#pragma unroll
            for (int c = 0; c < CT; ++c) red[(warp * K + r * KR + k) * COUT + ct * CT + c] = acc[k][c];
    __syncthreads();
    for (int i = threadIdx.x; i < K * COUT; i += 128) {
        float t = red[i];
#pragma unroll
        for (int wv = 1; wv < 4; ++wv) t += red[wv * K * COUT + i];
        partial[(long long)blockIdx.x * K * COUT + i] = t;
    }
}

inline bool a16(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; }

}  // namespace

bool stem_conv_supported(const ConvGeom& g) {
    return g.kh == 3 && g.kw == 3 && g.ph == 1 && g.pw == 1 && (g.stride == 1 || g.stride == 2) && g.Cin == 3 && (g.Cout == 32 || g.Cout == 64) &&
           (long long)g.N * g.Ho * g.Wo * g.Cout < (1LL << 40);
}

int stem_wgrad_blocks(const ConvGeom& g) {
    const long long chunks = ((long long)g.N * g.Ho * g.Wo + 31) / 32;
    const long long want = 4LL * sm_count();
    return (int)std::max<long long>(1, std::min<long long>(want, (chunks + 3) / 4));
}

size_t stem_wgrad_scratch_floats(const ConvGeom& g) { return stem_conv_supported(g) ? (size_t)stem_wgrad_blocks(g) * 27 * g.Cout : 0; }

template <typename T>
bool stem_conv_fwd(const T* x, const T* w, T* y, const ConvGeom& g, cudaStream_t st) {
    if (!stem_conv_supported(g) || !a16(y)) return false;
    const long long M = (long long)g.N * g.Ho * g.Wo;
    const dim3 grid((unsigned)((M + 127) / 128));
    if (g.Cout == 32) launch(stem_fwd_kernel<T, 3, 32>, grid, dim3(128), 0, st, x, w, y, g.N, g.H, g.W, g.Ho, g.Wo, g.stride);
    else launch(stem_fwd_kernel<T, 3, 64>, grid, dim3(128), 0, st, x, w, y, g.N, g.H, g.W, g.Ho, g.Wo, g.stride);
    return true;
}

template <typename T>
bool stem_conv_wgrad(const T* x, const T* dy, float* dw, float* scratch, const ConvGeom& g, cudaStream_t st) {
    if (!stem_conv_supported(g) || !scratch) return false;
    const int blocks = stem_wgrad_blocks(g);
    if (g.Cout == 32) launch(stem_wgrad_kernel<T, 3, 32>, dim3(blocks), dim3(128), 0, st, x, dy, scratch, g.N, g.H, g.W, g.Ho, g.Wo, g.stride);
    else launch(stem_wgrad_kernel<T, 3, 64>, dim3(blocks), dim3(128), 0, st, x, dy, scratch, g.N, g.H, g.W, g.Ho, g.Wo, g.stride);
    split_reduce_f32(scratch, blocks, 27LL * g.Cout, dw, st);
    return true;
}

template bool stem_conv_fwd<float>(const float*, const float*, float*, const ConvGeom&, cudaStream_t);
template bool stem_conv_fwd<__nv_bfloat16>(const __nv_bfloat16*, const __nv_bfloat16*, __nv_bfloat16*, const ConvGeom&, cudaStream_t);
template bool stem_conv_wgrad<float>(const float*, const float*, float*, float*, const ConvGeom&, cudaStream_t);
template bool stem_conv_wgrad<__nv_bfloat16>(const __nv_bfloat16*, const __nv_bfloat16*, float*, float*, const ConvGeom&, cudaStream_t);

}  // namespace ftp
