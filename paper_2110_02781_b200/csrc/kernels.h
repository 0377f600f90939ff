// Launchers of the device kernels.  Plain pointers and sizes; every launcher enqueues on the
// given stream and returns nothing: the caller checks cudaGetLastError().
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace ftp {

// A consumer may be handed the input of a batch norm instead of its output: it then applies
// z = min(max((y - mean) * scale + offset, lo), hi) to every element it loads (padding stays zero), so the
// normalised tensor never exists in memory.  mean is the float nearest the batch mean (subtracting it first keeps
// float accuracy in channels whose spread is small beside their mean), scale = gamma * rstd, and offset = beta minus
// the remainder of the mean times scale (formed in double by bn_finalize); one float per channel each, 16-byte
// aligned; (lo, hi) = (-inf, inf), (0, inf) or (0, 6).
struct BnXform {
    const float* mean;
    const float* scale;
    const float* offset;
    float lo, hi;
};
inline BnXform make_xform(const float* mean, const float* scale, const float* offset, int act) {
    const float inf = __builtin_huge_valf();
    return BnXform{mean, scale, offset, act == 0 ? -inf : 0.f, act == 2 ? 6.f : inf};
}

// Geometry of a (dense or depthwise) convolution.  Activations are (N, H, W, C).
struct ConvGeom {
    int N, H, W, Cin;     // input
    int Ho, Wo, Cout;     // output
    int kh, kw, stride, ph, pw;
};

// ---- fp32 SIMT contraction (gemm_f32.cu) ---------------------------------------------------
// y = act(conv(x, w) + bias) (+ addend): implicit GEMM, M = N*Ho*Wo, K = kh*kw*Cin.
// scratch (nullable): conv_gemm_scratch_floats(g) floats; lets small outputs split the reduction over blocks.
size_t conv_gemm_scratch_floats(const ConvGeom& g);
void conv_fwd_f32(const float* x, const float* w, const float* bias, float* y, float* scratch, const ConvGeom& g, int act,
                  cudaStream_t st);
// dx = conv^T(dy, w) (+ addend): implicit GEMM over the input pixels, K = kh*kw*Cout.
void conv_dgrad_f32(const float* dy, const float* w, const float* addend, float* dx, float* scratch, const ConvGeom& g,
                    cudaStream_t st);
// dw[kh][kw][cin][cout] = sum over output pixels; split over M with a fixed-order second pass.
// scratch must hold conv_wgrad_scratch_floats(g) floats.
size_t conv_wgrad_scratch_floats(const ConvGeom& g);
void conv_wgrad_f32(const float* x, const float* dy, float* dw, float* scratch, const ConvGeom& g, cudaStream_t st);

// the same kernels on bfloat16 tensors (bf16 weights, float accumulation, float weight gradient)
void conv_fwd_bf16_simt(const __nv_bfloat16* x, const __nv_bfloat16* w, const float* bias, __nv_bfloat16* y, const ConvGeom& g,
                        int act, cudaStream_t st);
void conv_dgrad_bf16_simt(const __nv_bfloat16* dy, const __nv_bfloat16* w, const __nv_bfloat16* addend, __nv_bfloat16* dx,
                          const ConvGeom& g, cudaStream_t st);
void conv_wgrad_bf16_simt(const __nv_bfloat16* x, const __nv_bfloat16* dy, float* dw, float* scratch, const ConvGeom& g,
                          cudaStream_t st);

// ---- tensor-core contraction (gemm_tc.cu): D[M,N] = A[M,K] * B[N,K]^T (+ addend), all bf16, both operands with K
// contiguous.  tc_gemm_supported: channel counts multiples of 8, 16-byte aligned pointers, driver entry point found.
// err: device int, stays 0 unless a bounded wait inside the kernel ran out.  Returns false if nothing was launched.
bool tc_gemm_supported(int M, int N, int K, const void* A, const void* B, const void* D, const void* addend);
// scratch (nullable): tc_gemm_scratch_floats(M, N, K) floats; lets products with few tiles and a long reduction cut it into slices
size_t tc_gemm_scratch_floats(int M, int N, int K);
bool tc_gemm_tn(const __nv_bfloat16* A, const __nv_bfloat16* B, const __nv_bfloat16* addend, __nv_bfloat16* D, float* scratch, int M, int N, int K,
                int* err, cudaStream_t st);
// 3x3 / stride 1 / pad 1 convolutions on the same kernels through 4-D tensor maps (zero fill = padding).
bool tc_conv3x3_supported(int N, int H, int W, int Ca, int No, const void* A, const void* B, const void* D, const void* addend);
bool tc_conv3x3(const __nv_bfloat16* A, const __nv_bfloat16* B, const __nv_bfloat16* addend, __nv_bfloat16* D, float* scratch, int N, int H, int W, int Ca,
                int No, int flip, int* err, cudaStream_t st);          // scratch: tc_gemm_scratch_floats(N*H*W, No, 9*Ca) floats, nullable
size_t tc_wgrad3x3_scratch_floats(long long R, int Mo, int No);
int tc_wgrad3x3(const __nv_bfloat16* X, const __nv_bfloat16* dY, float* dW, float* scratch, int N, int H, int W, int Mo, int No, int* err,
                cudaStream_t st);
size_t tc_wgrad_scratch_floats(long long R, int Mo, int No);
int tc_wgrad(const __nv_bfloat16* X, const __nv_bfloat16* dY, float* dW, float* scratch, long long R, int Mo, int No, int* err, cudaStream_t st);
void split_reduce_f32(const float* partial, int S, long long count, float* out, cudaStream_t st);   // out = sum over S partial arrays, in order

// ---- float contractions on tensor cores with split-tf32 arithmetic (gemm_tc32.cu); same conventions as above ----
bool tc32_supported(int M, int N, int K, const void* A, const void* B, const void* D, const void* addend);
// scratch (nullable): tc32_gemm_scratch_floats(M, N, K) floats; lets products with few tiles cut the reduction into slices
size_t tc32_gemm_scratch_floats(int M, int N, int K);
// B is [N][K]; B_lo (nullable): B - trunc_tf32(B) laid out like B, saves computing it per tile
struct ColStatsReq;
// a_xform (nullable): A holds the input of a batch norm that is applied to every tile as it is loaded
bool tc32_gemm(const float* A, const float* B, const float* B_lo, const float* addend, float* D, float* scratch, int M, int N, int K, int* err,
               cudaStream_t st, const ColStatsReq* stats = nullptr, const BnXform* a_xform = nullptr);
size_t tc32_wgrad_scratch_floats(long long R, int Mo, int No);
// dW[Mo][No] = X[R][Mo]^T dY[R][No], the fixed-order second pass over the reduction slices included
// x_xform (nullable): X holds the input of a batch norm that is applied as X is loaded
bool tc32_wgrad(const float* X, const float* dY, float* dW, float* scratch, long long R, int Mo, int No, int* err, cudaStream_t st,
                const BnXform* x_xform = nullptr);

// ---- first convolution of an image network (stem.cu): 3 x 3, pad 1, stride 1 or 2, 3 input channels, 32 or 64
// output channels, no bias or activation.  w is [3][3][3][cout] in T (float masters, or the bf16 shadow).
// false: shape not taken, nothing launched.
bool stem_conv_supported(const ConvGeom& g);
size_t stem_wgrad_scratch_floats(const ConvGeom& g);
template <typename T>
bool stem_conv_fwd(const T* x, const T* w, T* y, const ConvGeom& g, cudaStream_t st);
// dw [3][3][3][cout] float; scratch: stem_wgrad_scratch_floats(g) floats (one partial per block, added in block order)
template <typename T>
bool stem_conv_wgrad(const T* x, const T* dy, float* dw, float* scratch, const ConvGeom& g, cudaStream_t st);

// ---- streaming kernels (elem.cu); T = float or __nv_bfloat16, arithmetic in float ----------------
// Column reductions view a (M, C) tensor as (M/f, C*f) so that narrow tensors still fill whole
// 128-byte lines; `fold` picks f.  Partials are doubles: [chunks][2][C*f].
struct FoldPlan {
    int f;          // rows folded into one
    int cols;       // C * f
    int rows;       // M / f
    int chunks;     // row chunks (grid.y)
    int vec;        // elements per thread per row (16 bytes worth, or 1)
    // The reducing kernels merge the folded copies of a channel that fall inside one column tile, so a channel has
    // chunks * f / copies partial sums for the second pass to add.
    int fused;      // 1: merged layout in use (vectorisable tensor)
    int copies_fwd; // copies merged per column tile of 32 * vec columns (statistics kernel)
    int copies_bwd; // copies merged per column tile of 128 columns (backward reduction)
};
FoldPlan make_fold(long long M, int C, int elem_bytes);
// Scratch of the second pass: slice sums parked by its blocks and one ticket counter per channel group
// (and per tap for the depthwise gradient).  The counters must be zero before the first launch; every
// launch leaves them zero.  Launches sharing one FinScratch must be ordered on a stream.
struct FinScratch {
    double* part;
    unsigned* counters;
};
size_t fin_part_doubles(int C, int extra);      // extra = 9 for the depthwise weight gradient, else 1
size_t fin_counter_count(int C, int extra);
size_t fold_partial_doubles(const FoldPlan& fp);     // doubles needed for the partial sums

// Partial sums laid out [entries / fp][2][C * fp] (entry e: chunk e / fp, copy e % fp), as a reducing kernel leaves them.
struct PartialSums {
    const double* p;
    int entries, fp;
};
// A producer is asked to leave the statistics of its output for the batch norm that follows (fold = that batch
// norm's plan).  It stores what it wrote in *out; out->entries == 0 means it wrote none.
struct ColStatsReq {
    double* partial;
    const FoldPlan* fold;
    PartialSums* out;
};
size_t producer_partial_doubles(long long M, int C);      // room a producer may need: one entry per 128 rows
// D = sum of the S slices part[s][M][C] in slice order, and the statistics of D on the way.  false: nothing launched.
bool slice_sum_stats(const float* part, int S, float* D, long long M, int C, const FoldPlan& fp, double* partial, PartialSums* out, cudaStream_t st);
template <typename T>
PartialSums bn_stats(const T* y, long long M, int C, const FoldPlan& fp, double* partial, cudaStream_t st);
// mean/var -> scale (gamma * rstd), shift (a copy of beta), the mean as a two-float sum (mean + mean_lo),
// rstd; running statistics update (momentum, unbiased variance).  z = ((y - mean) - mean_lo) * scale + shift.
void bn_finalize(const PartialSums& ps, long long M, int C, const float* gamma,
                 const float* beta, float eps, float momentum, float* run_mean, float* run_var, float* scale,
                 float* shift, float* mean, float* mean_lo, float* rstd, float* offset, const FinScratch& fin, cudaStream_t st);
template <typename T>
void bn_apply(const T* y, const T* residual, T* z, long long M, int C, const FoldPlan& fp, const float* scale, const float* shift,
              const float* mean, const float* mean_lo, int act, cudaStream_t st);
// pass 1 of BN backward: sums of dz' and dz'*xhat with dz' = dz masked by the activation
template <typename T>
PartialSums bn_bwd_reduce(const T* dz, const T* y, long long M, int C, const FoldPlan& fp, const float* scale,
                   const float* shift, const float* mean, const float* mean_lo, const float* rstd, int act,
                   double* partial, cudaStream_t st);
// -> dgamma, dbeta and the per-channel coefficients coef[5][C]: a = gamma*rstd, then b = dbeta/M and
// c = dgamma/M each as a two-float sum (hi, lo)
void bn_bwd_finalize(const PartialSums& ps, long long M, int C, const float* gamma,
                     const float* rstd, float* dgamma, float* dbeta, float* coef, const FinScratch& fin, cudaStream_t st);
template <typename T>
void bn_bwd_apply(const T* dz, const T* y, const T* addend, T* dy, long long M, int C, const FoldPlan& fp, const float* scale,
                  const float* shift, const float* mean, const float* mean_lo, const float* rstd, const float* coef,
                  int act, cudaStream_t st);

// Backward of "act(pre + bias)": dpre = dout masked by the stored output; dbias = column sums.
// dpre may be NULL when act == 0 (then dpre == dout); dbias may be NULL.
template <typename T>
void act_bias_bwd(const T* dout, const T* out, T* dpre, long long M, int C, int act, const FoldPlan& fp,
                  double* partial, float* dbias, const FinScratch& fin, cudaStream_t st);
template <typename T>
void act_fwd(const T* x, T* y, long long n, int act, cudaStream_t st);
template <typename T>
void act_bwd(const T* dout, const T* x, const T* addend, T* dx, long long n, int act, cudaStream_t st);

template <typename T>
void dwconv_fwd(const T* x, const float* w, T* y, const ConvGeom& g, cudaStream_t st, const ColStatsReq* stats = nullptr, const BnXform* x_xform = nullptr);
template <typename T>
void dwconv_dgrad(const T* dy, const float* w, const T* addend, T* dx, const ConvGeom& g, cudaStream_t st);
size_t dwconv_wgrad_scratch_floats(const ConvGeom& g);
template <typename T>
void dwconv_wgrad(const T* x, const T* dy, float* dw, float* scratch, const ConvGeom& g, const FinScratch& fin, cudaStream_t st,
                  const BnXform* x_xform = nullptr);

// A kernel that produces the gradient with respect to the OUTPUT of a batch norm whose input it reads anyway may take
// over the first pass of that batch norm's backward: it stores the gradient masked by the activation and leaves the
// sums of g and g * xhat as partial sums (layout as the forward statistics) for bn_bwd_finalize.  *out: what it wrote
// (entries == 0: nothing; the separate reduction has to run).
struct BnBwdSumsReq {
    const float* rstd;       // per channel, 16-byte aligned
    double* partial;         // room: see the producer's *_stats_doubles
    PartialSums* out;
};
// Data gradient (+ addend) and weight gradient of a stride-1 depthwise convolution in one pass over dy (dx may be NULL).
// scratch: dwconv_wgrad_scratch_floats(g) floats.  false: shape not taken, nothing launched.
// sums (nullable, needs x_xform): x is the input of the batch norm before this convolution; see BnBwdSumsReq
// (partial: dwconv_bwd_stats_doubles(g) doubles).
size_t dwconv_bwd_stats_doubles(const ConvGeom& g);
template <typename T>
bool dwconv_bwd_fused(const T* x, const T* dy, const float* w, const T* addend, T* dx, float* dw, float* scratch, const ConvGeom& g, const FinScratch& fin,
                      cudaStream_t st, const BnXform* x_xform = nullptr, const BnBwdSumsReq* sums = nullptr, cudaStream_t fin_st = nullptr,
                      cudaEvent_t fin_fork = nullptr);
// fin_st (with fin_fork, an event of the caller): the kernel that adds the blocks' weight-gradient partials runs on that stream, after
// the main kernel (fin then belongs to that stream, and scratch must stay untouched until it has run)

template <typename T>
void maxpool_fwd(const T* x, T* y, int N, int H, int W, int C, cudaStream_t st);
template <typename T>
void maxpool_bwd(const T* dy, const T* x, T* dx, int N, int H, int W, int C, cudaStream_t st);
template <typename T>
void gap_fwd(const T* x, T* y, int N, int HW, int C, cudaStream_t st);
template <typename T>
void gap_bwd(const T* dy, T* dx, int N, int HW, int C, cudaStream_t st);

// loss = mean_n -log softmax(logits_n)[label_n]; dlogits = (softmax - onehot) / N.
// per_sample: float[N] scratch.  Labels outside [0, classes) contribute as if clamped.
void softmax_ce(const float* logits, const int32_t* labels, int N, int classes, float* per_sample,
                float* dlogits, float* loss, cudaStream_t st);

// Fused SGD: g += wd*w; m = first ? g : mu*m + g; w -= lr*m; optional bf16 shadow and snapshot stores.
// lo (nullable): receives w - trunc_tf32(w) of the updated weights.
void sgd_update(float* w, const float* g, float* m, long long n, float lr, float mu, float wd, int first,
                __nv_bfloat16* shadow, float* lo, float* snap_dev, float* snap_host, cudaStream_t st);
// dst = arithmetic mean of n (1..8) arrays, added in the order given
struct MeanSources { const float* p[8]; int n; };
void mean_f32(const MeanSources& src, float* dst, long long count, cudaStream_t st);
void tf32_lo(const float* w, float* lo, long long n, cudaStream_t st);                   // lo = w - trunc_tf32(w)
// Batched transposition of float matrices: entry e describes a [K][N] matrix at w + w_off whose transpose goes to
// wt + w_off ([N][K]) and the lo part of the transpose to wtl + w_off.  table: n + 1 device entries (the last one
// closes the tile range); tiles = table[n].tile0 - table[0].tile0 blocks are launched.
struct TransposeEntryDev { long long w_off; int K, N, tile0, taps; };       // taps: matrices of K x N one after the other (bf16 models: 9 for a 3x3 convolution)
void transpose_split_f32(const TransposeEntryDev* table, int n, int tile_base, int tiles, const float* w, float* wt, float* wtl, cudaStream_t st);
// bf16 models: wt[tap][N][K] = bf16(w[tap][K][N]) for n table entries in one launch (tiles: 32 x 32 tiles of all their matrices)
void transpose_bf16_batched(const TransposeEntryDev* table, int n, int tile_base, int tiles, const float* w, __nv_bfloat16* wt, cudaStream_t st);
void f32_to_bf16(const float* src, __nv_bfloat16* dst, long long n, cudaStream_t st);
void bf16_to_f32(const __nv_bfloat16* src, float* dst, long long n, cudaStream_t st);

int sm_count();

}  // namespace ftp
