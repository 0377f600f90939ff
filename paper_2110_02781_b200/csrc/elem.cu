// Streaming (HBM-bound) kernels: batch-norm statistics / apply / backward, activation and bias
// backward, depthwise 3x3 convolution, pooling, softmax cross-entropy and the fused SGD update.
// Every tensor is read and written with 16-byte accesses along the channel axis; every
// reduction runs in a fixed order (per-thread run, shared-memory column sum, then a second pass
// over the per-block partials) so results do not depend on scheduling.
#include <algorithm>
#include <cfloat>
#include <cstdlib>
#include <cstring>
#include <initializer_list>
#include "kernels.h"
#include "launch.cuh"
#include "bn_math.cuh"

namespace ftp {

bool pdl_enabled() {
    static int on = -1;
    if (on < 0) {
        const char* e = std::getenv("FTP_PDL");
        on = (e && std::strcmp(e, "0") == 0) ? 0 : 1;
    }
    return on == 1;
}

int sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
    }
    return n;
}

namespace {

// ---- 16-byte vector access with conversion to float ------------------------------------------
template <typename T> struct VecOf;
template <> struct VecOf<float> { static constexpr int N = 4; };
template <> struct VecOf<__nv_bfloat16> { static constexpr int N = 8; };

template <int V> __device__ __forceinline__ void ldv(const float* p, float (&o)[V]) {
    if constexpr (V == 4) { const float4 v = __ldg(reinterpret_cast<const float4*>(p)); o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w; }
    else { o[0] = __ldg(p); }
}
template <int V> __device__ __forceinline__ void ldv(const __nv_bfloat16* p, float (&o)[V]) {
    if constexpr (V == 8) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
        const unsigned u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) { o[2 * i] = __uint_as_float(u[i] << 16); o[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u); }
    } else if constexpr (V == 4) {
        const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
        o[0] = __uint_as_float(v.x << 16); o[1] = __uint_as_float(v.x & 0xffff0000u);
        o[2] = __uint_as_float(v.y << 16); o[3] = __uint_as_float(v.y & 0xffff0000u);
    } else { o[0] = __bfloat162float(*p); }
}
template <int V> __device__ __forceinline__ void ldplain(const float* p, float (&o)[V]) {       // coherent load of data the kernel also writes
    if constexpr (V == 4) { const float4 v = *reinterpret_cast<const float4*>(p); o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w; }
    else { o[0] = *p; }
}
template <int V> __device__ __forceinline__ void stv(float* p, const float (&v)[V]) {
    if constexpr (V == 4) *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
    else p[0] = v[0];
}
template <int V> __device__ __forceinline__ void stv(__nv_bfloat16* p, const float (&v)[V]) {
    if constexpr (V == 8) {
        unsigned u[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
            u[i] = *reinterpret_cast<const unsigned*>(&h);
        }
        *reinterpret_cast<uint4*>(p) = make_uint4(u[0], u[1], u[2], u[3]);
    } else if constexpr (V == 4) {
        const __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
        *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<const unsigned*>(&a), *reinterpret_cast<const unsigned*>(&b));
    } else { p[0] = __float2bfloat16_rn(v[0]); }
}
// V consecutive floats of a per-channel table (V is 1, 4 or 8; the address is 16-byte aligned for V >= 4)
template <int V> __device__ __forceinline__ void ldtab(const float* p, float (&o)[V]) {
    if constexpr (V == 1) o[0] = __ldg(p);
    else {
#pragma unroll
        for (int i = 0; i < V / 4; ++i) { const float4 v = __ldg(reinterpret_cast<const float4*>(p) + i); o[4 * i] = v.x; o[4 * i + 1] = v.y; o[4 * i + 2] = v.z; o[4 * i + 3] = v.w; }
    }
}

// Per-thread constants of a batch norm applied on load to V consecutive channels (see BnXform)
template <typename T, int V> struct XfRegs {
    float mu[V], sc[V], of[V];
    float lo, hi;
    __device__ __forceinline__ void load(const BnXform& x, int c) {
        ldtab<V>(x.mean + c, mu); ldtab<V>(x.scale + c, sc); ldtab<V>(x.offset + c, of);
        lo = x.lo; hi = x.hi;
    }
    __device__ __forceinline__ void apply(float (&v)[V]) const {
#pragma unroll
        for (int e = 0; e < V; ++e) v[e] = as_stored<T>(xf_z(v[e], mu[e], sc[e], of[e], lo, hi));
    }
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
inline unsigned flat_blocks(long long work, int threads) {
    long long b = (work + threads - 1) / threads;
    const long long cap = (long long)sm_count() * 16;
    if (b > cap) b = cap;
    if (b < 1) b = 1;
    return (unsigned)b;
}

// ---- folded column reductions --------------------------------------------------------------
// grid (column tiles of 32*V, row chunks); block (32, 8).  NS sums per column.
// copies > 1 (then copies * C == 32 * V): the copies of a channel inside the column tile are added up as well, in copy
// order, and the partial sums are laid out [chunk][NS][cols / copies].
template <typename T, int V, int NS>
__device__ __forceinline__ void fold_finish(float (&s)[NS][V], int cols, double* partial, int C, int copies);

template <typename T, int V, int NS, typename F>
__device__ __forceinline__ void fold_reduce(int rows, int cols, int rows_per_chunk, double* partial, F body, int C = 0, int copies = 1) {
    const int col = (blockIdx.x * 32 + threadIdx.x) * V;
    const int r0 = blockIdx.y * rows_per_chunk, r1 = min(rows, r0 + rows_per_chunk);
    float s[NS][V];
#pragma unroll
    for (int a = 0; a < NS; ++a)
#pragma unroll
        for (int e = 0; e < V; ++e) s[a][e] = 0.f;
    if (col < cols)
        for (int r = r0 + threadIdx.y; r < r1; r += 8) body((long long)r * cols + col, col, s);
    fold_finish<T, V, NS>(s, cols, partial, C, copies);
}

// The same reduction with the loads of two rows issued before either row is used: a thread that fetches 8 or 16
// bytes per tensor and row has too few bytes in flight to cover the memory latency otherwise (Little's law: four
// blocks of 256 threads per SM x 8 bytes x 2 tensors is 2.4 MB over the chip, a third of what 6.5 TB/s needs).
// The rows are still added in the order r, r + 8, r + 16, ..., so the sums are bit-identical to fold_reduce's.
template <typename T, int V, int NS, typename R, typename FL, typename FU>
__device__ __forceinline__ void fold_reduce2(int rows, int cols, int rows_per_chunk, double* partial, FL load, FU use, int C = 0, int copies = 1) {
    const int col = (blockIdx.x * 32 + threadIdx.x) * V;
    const int r0 = blockIdx.y * rows_per_chunk, r1 = min(rows, r0 + rows_per_chunk);
    float s[NS][V];
#pragma unroll
    for (int a = 0; a < NS; ++a)
#pragma unroll
        for (int e = 0; e < V; ++e) s[a][e] = 0.f;
    if (col < cols)
        for (int r = r0 + threadIdx.y; r < r1; r += 16) {
            R a, b;
            const bool two = r + 8 < r1;
            load((long long)r * cols + col, a);
            if (two) load((long long)(r + 8) * cols + col, b);
            use(a, s);
            if (two) use(b, s);
        }
    fold_finish<T, V, NS>(s, cols, partial, C, copies);
}

template <typename T, int V, int NS>
__device__ __forceinline__ void fold_finish(float (&s)[NS][V], int cols, double* partial, int C, int copies) {
    __shared__ float sh[NS][8][32 * V];
#pragma unroll
    for (int a = 0; a < NS; ++a)
#pragma unroll
        for (int e = 0; e < V; ++e) sh[a][threadIdx.y][threadIdx.x * V + e] = s[a][e];
    __syncthreads();
    if (copies > 1) {
        const int colsP = cols / copies;
        for (int q = threadIdx.y * 32 + threadIdx.x; q < NS * C; q += 256) {
            const int a = q / C, c = q - a * C;
            double t = 0.0;
            for (int k = 0; k < copies; ++k)
#pragma unroll
                for (int y = 0; y < 8; ++y) t += (double)sh[a][y][k * C + c];
            partial[((long long)blockIdx.y * NS + a) * colsP + blockIdx.x * C + c] = t;
        }
        return;
    }
    // 256 threads sum the 8 rows of NS * 32 * V columns in a fixed order
    for (int q = threadIdx.y * 32 + threadIdx.x; q < NS * 32 * V; q += 256) {
        const int a = q / (32 * V), c = q % (32 * V);
        const int gc = blockIdx.x * 32 * V + c;
        if (gc < cols) {
            double t = 0.0;
#pragma unroll
            for (int y = 0; y < 8; ++y) t += (double)sh[a][y][c];
            partial[((long long)blockIdx.y * NS + a) * cols + gc] = t;
        }
    }
}

// Second pass of every folded column reduction: sums over chunks and folded copies, one channel per x-lane.
// Grid (channel groups of FIN_X, G slices of the (chunk, copy) pairs, extra); block (FIN_X, FIN_Y).  Inside a block,
// y -> strided runs, four loads in flight at a time, then a fixed-shape tree over y in shared memory.  With
// G > 1 every block parks its slice sums in fin.part and takes a ticket; the block that draws the last ticket
// adds the G slice sums in slice order, so the result does not depend on which block that is.  Returns true in
// the block that holds the final sums (valid in its threads with y == 0).  NS consecutive sums from `first`.
constexpr int FIN_X = 8;
constexpr int FIN_Y = 128;
constexpr int FIN_GMAX = 16;
// FY: the block's extent in y, FIN_Y or FIN_Y_SMALL (few partial sums: a block of 1024 threads does not fit on an SM that
// also holds blocks of a kernel of the second stream, and would wait for them to leave).
constexpr int FIN_Y_SMALL = 32;
template <typename PT, int NS, int FY = FIN_Y>
__device__ __forceinline__ bool col_fold_sums(const PT* partial, int first, int ns, int chunks, int f, int C, int cols, int c,
                                              const FinScratch fin, double (&out)[NS]) {
    static_assert(FIN_X == 8 && (FY == 128 || FY == 32), "the reduction below is written for 8 x 128 or 8 x 32 threads");
    constexpr int WARPS = FIN_X * FY / 32;
    __shared__ double red[NS][WARPS][FIN_X];
    __shared__ unsigned ticket;
    double t[NS];
#pragma unroll
    for (int a = 0; a < NS; ++a) t[a] = 0.0;
    const int total = chunks * f, G = gridDim.y;
    const int per = (total + G - 1) / G, e0 = blockIdx.y * per, e1 = min(total, e0 + per);
    for (int e = e0 + threadIdx.y; e < e1; e += 4 * FY) {
        double v[NS][4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {                    // four independent loads in flight per sum
            const int ee = e + u * FY;
            const bool ok = ee < e1 && c < C;
            const int ch = ok ? ee / f : 0, k = ok ? ee - ch * f : 0;
#pragma unroll
            for (int a = 0; a < NS; ++a) v[a][u] = ok ? (double)partial[((long long)ch * ns + first + a) * cols + k * C + c] : 0.0;
        }
#pragma unroll
        for (int a = 0; a < NS; ++a) t[a] += (v[a][0] + v[a][1]) + (v[a][2] + v[a][3]);
    }
    // fixed-shape sum over y: the four y of a warp by shuffles, the warps through shared memory (a quarter of them per
    // lane group of the first warp, in order), the four lane groups by shuffles again
    const int lane = (threadIdx.y * FIN_X + threadIdx.x) & 31, warp = (threadIdx.y * FIN_X + threadIdx.x) >> 5;
#pragma unroll
    for (int a = 0; a < NS; ++a) {
        double v = t[a];
        v += __shfl_xor_sync(0xffffffffu, v, 8);
        v += __shfl_xor_sync(0xffffffffu, v, 16);
        if (lane < FIN_X) red[a][warp][lane] = v;
    }
    __syncthreads();
#pragma unroll
    for (int a = 0; a < NS; ++a) out[a] = 0.0;
    if (warp == 0) {
        const int x = lane & (FIN_X - 1), q = lane >> 3;
#pragma unroll
        for (int a = 0; a < NS; ++a) {
            double v = 0.0;
#pragma unroll
            for (int w = 0; w < WARPS / 4; ++w) v += red[a][q * (WARPS / 4) + w][x];
            v += __shfl_xor_sync(0xffffffffu, v, 8);
            v += __shfl_xor_sync(0xffffffffu, v, 16);
            out[a] = v;
        }
    }
    if (G == 1) return true;
    const int slot = blockIdx.z * gridDim.x + blockIdx.x;
    double* mine = fin.part + ((long long)slot * FIN_GMAX + blockIdx.y) * NS * FIN_X;
    if (threadIdx.y == 0)
#pragma unroll
        for (int a = 0; a < NS; ++a) mine[a * FIN_X + threadIdx.x] = out[a];
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0 && threadIdx.y == 0) ticket = atomicAdd(fin.counters + slot, 1u);
    __syncthreads();
    if (ticket != (unsigned)(G - 1)) return false;
    __threadfence();
    if (threadIdx.y == 0) {
#pragma unroll
        for (int a = 0; a < NS; ++a) {
            double r = 0.0;
            for (int g = 0; g < G; ++g) r += __ldcg(fin.part + ((long long)slot * FIN_GMAX + g) * NS * FIN_X + a * FIN_X + threadIdx.x);
            out[a] = r;
        }
        if (threadIdx.x == 0) fin.counters[slot] = 0u;       // ready for the next launch on this stream
    }
    return true;
}

template <typename T, int V>
__global__ void __launch_bounds__(256) bn_stats_kernel(const T* __restrict__ y, int rows, int cols, int rpc, double* __restrict__ partial, int C, int copies) {
    grid_dep_sync();
    fold_reduce<T, V, 2>(rows, cols, rpc, partial, [&](long long off, int, float (&s)[2][V]) {
        float v[V];
        ldv<V>(y + off, v);
#pragma unroll
        for (int e = 0; e < V; ++e) { s[0][e] += v[e]; s[1][e] = fmaf(v[e], v[e], s[1][e]); }
    }, C, copies);
}

// Second pass of a product whose reduction was cut into S slices, for an output that feeds a batch norm: adds the
// slices in slice order, stores the result and reduces its statistics on the way (same layout as bn_stats_kernel).
template <int V>
__global__ void __launch_bounds__(256) slice_sum_stats_kernel(const float* __restrict__ part, int S, long long slice_elems, float* __restrict__ out,
                                                              int rows, int cols, int rpc, double* __restrict__ partial, int C, int copies) {
    grid_dep_sync();
    fold_reduce<float, V, 2>(rows, cols, rpc, partial, [&](long long off, int, float (&s)[2][V]) {
        float a[V];
        ldv<V>(part + off, a);
        for (int z = 1; z < S; ++z) {
            float v[V];
            ldv<V>(part + (long long)z * slice_elems + off, v);
#pragma unroll
            for (int e = 0; e < V; ++e) a[e] += v[e];
        }
        stv<V>(out + off, a);
#pragma unroll
        for (int e = 0; e < V; ++e) { s[0][e] += a[e]; s[1][e] = fmaf(a[e], a[e], s[1][e]); }
    }, C, copies);
}

// 1 / sqrt(v) in double from the float estimate and two Newton steps (the divide-and-root sequence is several
// hundred cycles of dependent fp64 work on a kernel that is nothing but latency)
__device__ __forceinline__ double rsqrt_f64(double v) {
    double r = (double)rsqrtf((float)v);
    r = r * (1.5 - 0.5 * v * r * r);
    r = r * (1.5 - 0.5 * v * r * r);
    return r;
}

template <int FY>
__global__ void __launch_bounds__(FIN_X * FY) bn_finalize_kernel(const double* __restrict__ partial, int chunks, int f, int C, int cols, double M, double inv_M, double unbias,
                                   const float* __restrict__ gamma, const float* __restrict__ beta, float eps, float mom,
                                   float* run_mean, float* run_var, float* scale, float* shift, float* mean, float* mean_lo, float* rstd,
                                   float* offset, const FinScratch fin) {
    grid_dep_sync();
    const int c = blockIdx.x * FIN_X + threadIdx.x;
    float ga = 0.f, be = 0.f, rm = 0.f, rv = 0.f;                    // fetched up front: their latency hides behind the sums
    if (threadIdx.y == 0 && c < C) { ga = gamma[c]; be = beta[c]; rm = run_mean[c]; rv = run_var[c]; }
    double ss[2];
    if (!col_fold_sums<double, 2, FY>(partial, 0, 2, chunks, f, C, cols, c, fin, ss)) return;
    const double s1 = ss[0], s2 = ss[1];
    if (threadIdx.y == 0 && c < C) {
        const double mu = s1 * inv_M;
        double var = s2 * inv_M - mu * mu;
        if (var < 0.0) var = 0.0;
        const double rs = rsqrt_f64(var + (double)eps);
        const float sc = (float)((double)ga * rs);
        scale[c] = sc;
        offset[c] = (float)((double)be - (mu - (double)(float)mu) * (double)sc);     // z = (y - mean) * scale + offset, for readers that normalise as they load
        shift[c] = be;                            // z = (y - mean) * scale + beta, the mean kept as a two-float sum
        const float mh = (float)mu;
        mean[c] = mh;
        mean_lo[c] = (float)(mu - (double)mh);
        rstd[c] = (float)rs;
        run_mean[c] = (float)((1.0 - (double)mom) * (double)rm + (double)mom * mu);
        run_var[c] = (float)((1.0 - (double)mom) * (double)rv + (double)mom * (var * unbias));
    }
}

// z = act(((y - mean) - mean_lo) * scale + shift) (+ residual) on the folded view: grid (column tiles, row chunks),
// block (32, 8).  A thread keeps the constants of its V channels in registers and walks the rows of its chunk, so
// the only memory traffic per element is the streamed tensors themselves.
template <typename T, int V>
__global__ void __launch_bounds__(256) bn_apply_kernel(const T* __restrict__ y, const T* __restrict__ res, T* __restrict__ z,
                                                       int rows, int cols, int rpc, int C, const float* __restrict__ scale,
                                                       const float* __restrict__ shift, const float* __restrict__ mean,
                                                       const float* __restrict__ mean_lo, int act) {
    grid_dep_sync();
    const int col = (blockIdx.x * 32 + threadIdx.x) * V;
    if (col >= cols) return;
    const int c = col % C;
    float sc[V], sh[V], mu[V], ml[V];
    ldtab<V>(scale + c, sc); ldtab<V>(shift + c, sh); ldtab<V>(mean + c, mu); ldtab<V>(mean_lo + c, ml);
    const int r0 = blockIdx.y * rpc, r1 = min(rows, r0 + rpc);
    for (int r = r0 + threadIdx.y; r < r1; r += 8) {
        const long long off = (long long)r * cols + col;
        float v[V];
        ldv<V>(y + off, v);
#pragma unroll
        for (int e = 0; e < V; ++e) v[e] = act_f(bn_z(v[e], mu[e], ml[e], sc[e], sh[e]), act);
        if (res) {
            float q[V];
            ldv<V>(res + off, q);
#pragma unroll
            for (int e = 0; e < V; ++e) v[e] += q[e];
        }
        stv<V>(z + off, v);
    }
}

template <typename T, int V>
__global__ void __launch_bounds__(256) bn_bwd_reduce_kernel(const T* __restrict__ dz, const T* __restrict__ y, int rows, int cols, int rpc, int C,
                                                            const float* __restrict__ scale, const float* __restrict__ shift,
                                                            const float* __restrict__ mean, const float* __restrict__ mean_lo,
                                                            const float* __restrict__ rstd, int act, double* __restrict__ partial, int copies) {
    grid_dep_sync();
    const int col = (blockIdx.x * 32 + threadIdx.x) * V;
    float sc[V], sh[V], mu[V], ml[V], rs[V];
    if (col < cols) { const int c = col % C; ldtab<V>(scale + c, sc); ldtab<V>(shift + c, sh); ldtab<V>(mean + c, mu); ldtab<V>(mean_lo + c, ml); ldtab<V>(rstd + c, rs); }
    struct Row { float d[V], v[V]; };
    fold_reduce2<T, V, 2, Row>(rows, cols, rpc, partial,
        [&](long long off, Row& q) { ldv<V>(dz + off, q.d); ldv<V>(y + off, q.v); },
        [&](const Row& q, float (&s)[2][V]) {
#pragma unroll
            for (int e = 0; e < V; ++e) {
                const float g = act_pass(bn_z(q.v[e], mu[e], ml[e], sc[e], sh[e]), act) ? q.d[e] : 0.f;
                s[0][e] += g;
                s[1][e] = fmaf(g, ((q.v[e] - mu[e]) - ml[e]) * rs[e], s[1][e]);
            }
        }, C, copies);
}

template <int FY>
__global__ void __launch_bounds__(FIN_X * FY) bn_bwd_finalize_kernel(const double* __restrict__ partial, int chunks, int f, int C, int cols, double inv_M,
                                       const float* __restrict__ gamma, const float* __restrict__ rstd, float* dgamma,
                                       float* dbeta, float* coef, const FinScratch fin) {
    grid_dep_sync();
    const int c = blockIdx.x * FIN_X + threadIdx.x;
    float ga = 0.f, rs = 0.f;
    if (threadIdx.y == 0 && c < C) { ga = gamma[c]; rs = rstd[c]; }
    double ss[2];
    if (!col_fold_sums<double, 2, FY>(partial, 0, 2, chunks, f, C, cols, c, fin, ss)) return;
    const double s1 = ss[0], s2 = ss[1];
    if (threadIdx.y == 0 && c < C) {
        dbeta[c] = (float)s1;
        dgamma[c] = (float)s2;
        coef[c] = ga * rs;
        const double b = s1 * inv_M, cc = s2 * inv_M;      // kept as two-float sums: they are subtracted from values of their own size
        const float bh = (float)b, ch = (float)cc;
        coef[C + c] = bh; coef[2 * C + c] = (float)(b - (double)bh);
        coef[3 * C + c] = ch; coef[4 * C + c] = (float)(cc - (double)ch);
    }
}

// dy = a * ((g - b) - xhat * c) (+ addend), g = dz masked by the activation; same thread layout as bn_apply_kernel
template <typename T, int V>
__global__ void __launch_bounds__(256) bn_bwd_apply_kernel(const T* __restrict__ dz, const T* __restrict__ y, const T* __restrict__ addend,
                                                           T* __restrict__ dy, int rows, int cols, int rpc, int C, const float* __restrict__ scale,
                                                           const float* __restrict__ shift, const float* __restrict__ mean,
                                                           const float* __restrict__ mean_lo, const float* __restrict__ rstd,
                                                           const float* __restrict__ coef, int act) {
    grid_dep_sync();
    const int col = (blockIdx.x * 32 + threadIdx.x) * V;
    if (col >= cols) return;
    const int c = col % C;
    float sc[V], sh[V], mu[V], ml[V], rs[V], ca[V], bh[V], bl[V], ch[V], cl[V];
    ldtab<V>(scale + c, sc); ldtab<V>(shift + c, sh); ldtab<V>(mean + c, mu); ldtab<V>(mean_lo + c, ml); ldtab<V>(rstd + c, rs);
    ldtab<V>(coef + c, ca); ldtab<V>(coef + C + c, bh); ldtab<V>(coef + 2 * C + c, bl);
    ldtab<V>(coef + 3 * C + c, ch); ldtab<V>(coef + 4 * C + c, cl);
    const int r0 = blockIdx.y * rpc, r1 = min(rows, r0 + rpc);
    // two rows per trip, all their loads issued before the first use (see fold_reduce2)
    for (int r = r0 + threadIdx.y; r < r1; r += 16) {
        const bool two = r + 8 < r1;
        const long long off[2] = {(long long)r * cols + col, (long long)(r + 8) * cols + col};
        float d[2][V], v[2][V], a[2][V];
#pragma unroll
        for (int k = 0; k < 2; ++k)
            if (k == 0 || two) {
                ldv<V>(dz + off[k], d[k]);
                ldv<V>(y + off[k], v[k]);
                if (addend) ldv<V>(addend + off[k], a[k]);
            }
#pragma unroll
        for (int k = 0; k < 2; ++k)
            if (k == 0 || two) {
                float o[V];
#pragma unroll
                for (int e = 0; e < V; ++e) {
                    const float cen = (v[k][e] - mu[e]) - ml[e];
                    const float g = act_pass(fmaf(cen, sc[e], sh[e]), act) ? d[k][e] : 0.f;
                    const float xh = cen * rs[e];
                    float t = (g - bh[e]) - bl[e];
                    t = fmaf(-xh, ch[e], t);
                    t = fmaf(-xh, cl[e], t);
                    o[e] = ca[e] * t;
                    if (addend) o[e] += a[k][e];
                }
                stv<V>(dy + off[k], o);
            }
    }
}

template <typename T, int V>
__global__ void __launch_bounds__(256) act_bias_bwd_kernel(const T* __restrict__ dout, const T* __restrict__ out, T* __restrict__ dpre,
                                                           int rows, int cols, int rpc, int act, double* __restrict__ partial) {
    grid_dep_sync();
    fold_reduce<T, V, 1>(rows, cols, rpc, partial, [&](long long off, int, float (&s)[1][V]) {
        float d[V];
        ldv<V>(dout + off, d);
        if (act != 0) {
            float o[V];
            ldv<V>(out + off, o);
#pragma unroll
            for (int e = 0; e < V; ++e) d[e] = act_pass(o[e], act) ? d[e] : 0.f;
        }
        if (dpre) stv<V>(dpre + off, d);
#pragma unroll
        for (int e = 0; e < V; ++e) s[0][e] += d[e];
    });
}

__global__ void colsum_finalize_kernel(const double* __restrict__ partial, int chunks, int f, int C, int cols, float* out, const FinScratch fin) {
    grid_dep_sync();
    const int c = blockIdx.x * FIN_X + threadIdx.x;
    double ss[1];
    if (!col_fold_sums<double, 1>(partial, 0, 1, chunks, f, C, cols, c, fin, ss)) return;
    if (threadIdx.y == 0 && c < C) out[c] = (float)ss[0];
}

template <typename T, int V>
__global__ void __launch_bounds__(256) act_fwd_kernel(const T* __restrict__ x, T* __restrict__ y, long long nvec, int act) {
    grid_dep_sync();
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += (long long)gridDim.x * blockDim.x) {
        float v[V];
        ldv<V>(x + i * V, v);
#pragma unroll
        for (int e = 0; e < V; ++e) v[e] = act_f(v[e], act);
        stv<V>(y + i * V, v);
    }
}

template <typename T, int V>
__global__ void __launch_bounds__(256) act_bwd_kernel(const T* __restrict__ dout, const T* __restrict__ x, const T* __restrict__ addend,
                                                      T* __restrict__ dx, long long nvec, int act) {
    grid_dep_sync();
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += (long long)gridDim.x * blockDim.x) {
        float d[V], v[V];
        ldv<V>(dout + i * V, d);
        ldv<V>(x + i * V, v);
#pragma unroll
        for (int e = 0; e < V; ++e) d[e] = act_pass(v[e], act) ? d[e] : 0.f;
        if (addend) {
            float a[V];
            ldv<V>(addend + i * V, a);
#pragma unroll
            for (int e = 0; e < V; ++e) d[e] += a[e];
        }
        stv<V>(dx + i * V, d);
    }
}

// ---- depthwise 3x3 ------------------------------------------------------------------------------
// The two gather kernels below map a block of 256 threads onto a tile of 64 output pixels (TW = 2^tws wide,
// 64 / TW rows of the (image, row) index space) times 8 channel vectors, two pixels per thread, so that the
// nine taps of neighbouring outputs hit the lines their neighbours just fetched.  grid (pixel tiles, ceil(CV / 8)).
template <typename T, int V, bool XF>
__global__ void __launch_bounds__(256) dw_fwd_kernel(const T* __restrict__ x, const float* __restrict__ w, T* __restrict__ y, ConvGeom g, int tws, BnXform xf) {
    grid_dep_sync();
    const int CV = g.Cin / V;
    const int cv = blockIdx.y * 8 + (threadIdx.x & 7);
    if (cv >= CV) return;
    const int c = cv * V;
    XfRegs<T, V> xr;
    if constexpr (XF) xr.load(xf, c);
    const int slot = threadIdx.x >> 3, TW = 1 << tws, half = 32 >> tws;
    const int tiles_w = (g.Wo + TW - 1) >> tws;
    const int tw_i = blockIdx.x % tiles_w, tr_i = blockIdx.x / tiles_w;
    const int wo = tw_i * TW + (slot & (TW - 1));
    if (wo >= g.Wo) return;
    const int rows = g.N * g.Ho;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int R = tr_i * 2 * half + (slot >> tws) + k * half;
        if (R >= rows) break;
        const int n = R / g.Ho, ho = R - n * g.Ho;
        const long long i = ((long long)R * g.Wo + wo) * CV + cv;
        float acc[V];
#pragma unroll
        for (int e = 0; e < V; ++e) acc[e] = 0.f;
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            const int hi = ho * g.stride - g.ph + r;
            if (hi < 0 || hi >= g.H) continue;
#pragma unroll
            for (int s = 0; s < 3; ++s) {
                const int wi = wo * g.stride - g.pw + s;
                if (wi < 0 || wi >= g.W) continue;
                float v[V], k[V];
                ldv<V>(x + ((long long)(n * g.H + hi) * g.W + wi) * g.Cin + c, v);
                if constexpr (XF) xr.apply(v);
                ldtab<V>(w + (r * 3 + s) * g.Cin + c, k);
#pragma unroll
                for (int e = 0; e < V; ++e) acc[e] = fmaf(v[e], k[e], acc[e]);
            }
        }
        stv<V>(y + i * V, acc);
    }
}

// STRIDE is a compile-time 1 or 2 (0: read g.stride): the gather divides by it once per tap, and a division by a
// run-time value costs more than the tap's multiply-adds.
template <typename T, int V, int STRIDE>
__global__ void __launch_bounds__(256) dw_dgrad_kernel(const T* __restrict__ dy, const float* __restrict__ w, const T* __restrict__ addend,
                                                       T* __restrict__ dx, ConvGeom g, int tws) {
    grid_dep_sync();
    const int CV = g.Cin / V;
    const int cv = blockIdx.y * 8 + (threadIdx.x & 7);
    if (cv >= CV) return;
    const int c = cv * V;
    const int slot = threadIdx.x >> 3, TW = 1 << tws, half = 32 >> tws;
    const int tiles_w = (g.W + TW - 1) >> tws;
    const int tw_i = blockIdx.x % tiles_w, tr_i = blockIdx.x / tiles_w;
    const int wi = tw_i * TW + (slot & (TW - 1));
    if (wi >= g.W) return;
    const int rows = g.N * g.H;
    const int stride = STRIDE > 0 ? STRIDE : g.stride;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int R = tr_i * 2 * half + (slot >> tws) + k * half;
        if (R >= rows) break;
        const int n = R / g.H, hi = R - n * g.H;
        const long long i = ((long long)R * g.W + wi) * CV + cv;
        float acc[V];
#pragma unroll
        for (int e = 0; e < V; ++e) acc[e] = 0.f;
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            const int th = hi + g.ph - r;
            if (th < 0) continue;
            const int ho = th / stride;
            if (ho * stride != th || ho >= g.Ho) continue;
#pragma unroll
            for (int s = 0; s < 3; ++s) {
                const int tw = wi + g.pw - s;
                if (tw < 0) continue;
                const int wo = tw / stride;
                if (wo * stride != tw || wo >= g.Wo) continue;
                float v[V], k[V];
                ldv<V>(dy + ((long long)(n * g.Ho + ho) * g.Wo + wo) * g.Cin + c, v);
                ldtab<V>(w + (r * 3 + s) * g.Cin + c, k);
#pragma unroll
                for (int e = 0; e < V; ++e) acc[e] = fmaf(v[e], k[e], acc[e]);
            }
        }
        if (addend) {
            float a[V];
            ldv<V>(addend + i * V, a);
#pragma unroll
            for (int e = 0; e < V; ++e) acc[e] += a[e];
        }
        stv<V>(dx + i * V, acc);
    }
}

// Stride-1 depthwise 3x3 (padding 1), forward (FLIP = 0) or data gradient (FLIP = 1: the same sum with the
// taps mirrored): a thread computes four neighbouring outputs of one row for one channel vector from the
// 3 x 6 inputs they share, so every input vector is loaded once per row of taps instead of three times and
// the six loads of a row are in flight together.  Block: 8 channel vectors x 32 strips; strips are numbered
// row-major over (image, row, strip of 4 columns).
template <typename T, int V, int FLIP, bool STATS, bool XF>
__device__ __forceinline__ void dw_strip_body(const T* __restrict__ x, const float* __restrict__ w, const T* __restrict__ addend, T* __restrict__ y,
                                              int H, int W, int C, int c, long long strip, int strips_w, float (&su)[V], float (&sq)[V],
                                              const XfRegs<T, V>& xr) {
    const int w0 = (int)(strip % strips_w) * 4;
    const long long R = strip / strips_w;                 // image * H + row
    const int h = (int)(R % H);
    float acc[4][V];
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int e = 0; e < V; ++e) acc[j][e] = 0.f;
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        const int hi = h - 1 + r;
        if (hi < 0 || hi >= H) continue;
        const T* row = x + ((R - h + hi) * W) * (long long)C + c;
        float in[6][V];
#pragma unroll
        for (int j = 0; j < 6; ++j) {
            const int wi = w0 - 1 + j;
            if (wi >= 0 && wi < W) {
                ldv<V>(row + (long long)wi * C, in[j]);
                if constexpr (XF) xr.apply(in[j]);
            } else {
#pragma unroll
                for (int e = 0; e < V; ++e) in[j][e] = 0.f;
            }
        }
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            float k[V];
            ldtab<V>(w + ((FLIP ? 2 - r : r) * 3 + (FLIP ? 2 - s : s)) * C + c, k);
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int e = 0; e < V; ++e) acc[j][e] = fmaf(in[j + s][e], k[e], acc[j][e]);
        }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (w0 + j >= W) break;
        const long long o = ((R * W) + w0 + j) * (long long)C + c;
        if (addend) {
            float a[V];
            ldv<V>(addend + o, a);
#pragma unroll
            for (int e = 0; e < V; ++e) acc[j][e] += a[e];
        }
        stv<V>(y + o, acc[j]);
        if constexpr (STATS) {
#pragma unroll
            for (int e = 0; e < V; ++e) { const float v = as_stored<T>(acc[j][e]); su[e] += v; sq[e] = fmaf(v, v, sq[e]); }
        }
    }
}

// STATS: the block also leaves the column sums and sums of squares of the values it stored (as stored: rounded to T)
// in stats[blockIdx.x][2][C], for the batch norm that follows.
template <typename T, int V, int FLIP, int STATS, bool XF>
__global__ void __launch_bounds__(256) dw_strip_kernel(const T* __restrict__ x, const float* __restrict__ w, const T* __restrict__ addend,
                                                       T* __restrict__ y, int N, int H, int W, int C, double* __restrict__ stats, BnXform xf) {
    grid_dep_sync();
    const int CV = C / V;
    const int cv = blockIdx.y * 8 + (threadIdx.x & 7);
    const int c = cv * V;
    const int strips_w = (W + 3) >> 2;
    const long long strip = (long long)blockIdx.x * 32 + (threadIdx.x >> 3);
    const bool live = cv < CV && strip < (long long)N * H * strips_w;
    XfRegs<T, V> xr;
    if constexpr (XF) { if (cv < CV) xr.load(xf, c); }
    if constexpr (STATS) {
        __shared__ float shs[2][32][8 * V];
        float su[V], sq[V];
#pragma unroll
        for (int e = 0; e < V; ++e) su[e] = sq[e] = 0.f;
        if (live) dw_strip_body<T, V, FLIP, true, XF>(x, w, addend, y, H, W, C, c, strip, strips_w, su, sq, xr);
#pragma unroll
        for (int e = 0; e < V; ++e) { shs[0][threadIdx.x >> 3][(threadIdx.x & 7) * V + e] = su[e]; shs[1][threadIdx.x >> 3][(threadIdx.x & 7) * V + e] = sq[e]; }
        __syncthreads();
        if (threadIdx.x < 2 * 8 * V) {
            const int a = threadIdx.x / (8 * V), ch = threadIdx.x % (8 * V), gc = blockIdx.y * 8 * V + ch;
            if (gc < C) {
                double t = 0.0;
#pragma unroll
                for (int k = 0; k < 32; ++k) t += (double)shs[a][k][ch];
                stats[((long long)blockIdx.x * 2 + a) * C + gc] = t;
            }
        }
    } else {
        float su[V], sq[V];
        if (live) dw_strip_body<T, V, FLIP, false, XF>(x, w, addend, y, H, W, C, c, strip, strips_w, su, sq, xr);
    }
}

// Depthwise weight gradient on the folded view: grid (column tiles of 32*V, pixel-row chunks), block (32, 8).
// A thread owns V folded columns (a fixed channel vector and a fixed pixel offset within each folded row)
// and walks the rows of its chunk; the 9 taps are reduced over y three at a time through shared memory.
// partial[chunk][9][cols] (float).
template <typename T, int V, bool XF>
__global__ void __launch_bounds__(256) dw_wgrad_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ partial, ConvGeom g,
                                                       int rows, int cols, int f, int rpc, BnXform xf) {
    grid_dep_sync();
    __shared__ float sh[3][8][32 * V];
    const int col = (blockIdx.x * 32 + threadIdx.x) * V;
    const int r0 = blockIdx.y * rpc, r1 = min(rows, r0 + rpc);
    float acc[9][V];
#pragma unroll
    for (int t = 0; t < 9; ++t)
#pragma unroll
        for (int e = 0; e < V; ++e) acc[t][e] = 0.f;
    if (col < cols) {
        const int kf = col / g.Cin, c = col - kf * g.Cin;        // pixel offset inside a folded row, channel
        XfRegs<T, V> xr;
        if constexpr (XF) xr.load(xf, c);
        for (int r = r0 + threadIdx.y; r < r1; r += 8) {
            const long long pix = (long long)r * f + kf;
            const int wo = (int)(pix % g.Wo);
            const long long q = pix / g.Wo;
            const int ho = (int)(q % g.Ho), n = (int)(q / g.Ho);
            float d[V];
            ldv<V>(dy + pix * g.Cin + c, d);
#pragma unroll
            for (int rr = 0; rr < 3; ++rr) {
                const int hi = ho * g.stride - g.ph + rr;
                if (hi < 0 || hi >= g.H) continue;
#pragma unroll
                for (int ss = 0; ss < 3; ++ss) {
                    const int wi = wo * g.stride - g.pw + ss;
                    if (wi < 0 || wi >= g.W) continue;
                    float v[V];
                    ldv<V>(x + ((long long)(n * g.H + hi) * g.W + wi) * g.Cin + c, v);
                    if constexpr (XF) xr.apply(v);
#pragma unroll
                    for (int e = 0; e < V; ++e) acc[rr * 3 + ss][e] = fmaf(v[e], d[e], acc[rr * 3 + ss][e]);
                }
            }
        }
    }
#pragma unroll
    for (int gq = 0; gq < 3; ++gq) {
        __syncthreads();
#pragma unroll
        for (int t = 0; t < 3; ++t)
#pragma unroll
            for (int e = 0; e < V; ++e) sh[t][threadIdx.y][threadIdx.x * V + e] = acc[gq * 3 + t][e];
        __syncthreads();
        for (int q = threadIdx.y * 32 + threadIdx.x; q < 3 * 32 * V; q += 256) {
            const int t = q / (32 * V), cc = q % (32 * V);
            const int gc = blockIdx.x * 32 * V + cc;
            if (gc < cols) {
                float sum = 0.f;
#pragma unroll
                for (int y = 0; y < 8; ++y) sum += sh[t][y][cc];
                partial[((long long)blockIdx.y * 9 + gq * 3 + t) * cols + gc] = sum;
            }
        }
    }
}

// Stride-1 depthwise weight gradient (padding 1) on strips of four neighbouring outputs, as dw_strip_kernel: a
// thread loads the four output gradients and the 3 x 6 inputs of a strip once and feeds all nine taps from them;
// it walks strips blockIdx.x * 32 + slot, + gridDim.x * 32, ... with its nine accumulators in registers, and the
// 32 strip slots of the block are added in slot order through shared memory.  partial[blockIdx.x][9][C] (float).
template <typename T, int V, bool XF>
__global__ void __launch_bounds__(256) dw_wgrad_strip_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ partial, int N, int H,
                                                             int W, int C, BnXform xf) {
    grid_dep_sync();
    __shared__ float sh[3][32][8 * V];
    const int CV = C / V, cvl = threadIdx.x & 7, cv = blockIdx.y * 8 + cvl, slot = threadIdx.x >> 3;
    const int c = cv * V;
    const int strips_w = (W + 3) >> 2;
    const long long strips = (long long)N * H * strips_w;
    float acc[9][V];
#pragma unroll
    for (int t = 0; t < 9; ++t)
#pragma unroll
        for (int e = 0; e < V; ++e) acc[t][e] = 0.f;
    if (cv < CV) {
        XfRegs<T, V> xr;
        if constexpr (XF) xr.load(xf, c);
        for (long long s = (long long)blockIdx.x * 32 + slot; s < strips; s += (long long)gridDim.x * 32) {
            const int w0 = (int)(s % strips_w) * 4;
            const long long R = s / strips_w;
            const int h = (int)(R % H);
            float d[4][V];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (w0 + j < W) ldv<V>(dy + ((R * W) + w0 + j) * (long long)C + c, d[j]);
                else {
#pragma unroll
                    for (int e = 0; e < V; ++e) d[j][e] = 0.f;
                }
            }
#pragma unroll
            for (int rr = 0; rr < 3; ++rr) {
                const int hi = h - 1 + rr;
                if (hi < 0 || hi >= H) continue;
                const T* row = x + ((R - h + hi) * W) * (long long)C + c;
                float in[6][V];
#pragma unroll
                for (int j = 0; j < 6; ++j) {
                    const int wi = w0 - 1 + j;
                    if (wi >= 0 && wi < W) {
                        ldv<V>(row + (long long)wi * C, in[j]);
                        if constexpr (XF) xr.apply(in[j]);
                    } else {
#pragma unroll
                        for (int e = 0; e < V; ++e) in[j][e] = 0.f;
                    }
                }
#pragma unroll
                for (int ss = 0; ss < 3; ++ss)
#pragma unroll
                    for (int j = 0; j < 4; ++j)
#pragma unroll
                        for (int e = 0; e < V; ++e) acc[rr * 3 + ss][e] = fmaf(in[j + ss][e], d[j][e], acc[rr * 3 + ss][e]);
            }
        }
    }
#pragma unroll
    for (int gq = 0; gq < 3; ++gq) {
        __syncthreads();
#pragma unroll
        for (int t = 0; t < 3; ++t)
#pragma unroll
            for (int e = 0; e < V; ++e) sh[t][slot][cvl * V + e] = acc[gq * 3 + t][e];
        __syncthreads();
        for (int q = threadIdx.x; q < 3 * 8 * V; q += 256) {
            const int t = q / (8 * V), cc = q % (8 * V);
            const int gc = blockIdx.y * 8 * V + cc;
            if (gc < C) {
                float sum = 0.f;
#pragma unroll 8
                for (int y = 0; y < 32; ++y) sum += sh[t][y][cc];
                partial[((long long)blockIdx.x * 9 + gq * 3 + t) * C + gc] = sum;
            }
        }
    }
}

// The same weight gradient with three threads per strip, one per filter row (used for bf16 tensors, where it is
// 20 % faster; float tensors are 10 % faster with the kernel above): a thread loads the four output gradients and the six inputs of its row once and feeds
// its three taps from them.  (One thread per strip with all nine taps kept 36 accumulators and 109 registers: two
// blocks per SM and a kernel that waited on its loads.)  Block: 8 channel vectors x 32 slots, slot = 3 * strip + row
// for 10 strips, two slots idle; a block walks strips blockIdx.x * 10 + k, + gridDim.x * 10, ... and adds its slots
// in slot order through shared memory.  partial[blockIdx.x][9][C] (float).
constexpr int DW_WG_STRIPS = 10;
template <typename T, int V, bool XF>
__global__ void __launch_bounds__(256) dw_wgrad_rows_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ partial, int N, int H,
                                                             int W, int C, BnXform xf) {
    grid_dep_sync();
    __shared__ float sh[3][32][8 * V];
    const int CV = C / V, cvl = threadIdx.x & 7, cv = blockIdx.y * 8 + cvl, slot = threadIdx.x >> 3;
    const int c = cv * V;
    const int k = slot / 3, rr = slot - 3 * k;              // strip within the block's group of ten, filter row
    const int strips_w = (W + 3) >> 2;
    const long long strips = (long long)N * H * strips_w;
    float acc[3][V];
#pragma unroll
    for (int t = 0; t < 3; ++t)
#pragma unroll
        for (int e = 0; e < V; ++e) acc[t][e] = 0.f;
    if (cv < CV && k < DW_WG_STRIPS) {
        XfRegs<T, V> xr;
        if constexpr (XF) xr.load(xf, c);
        for (long long s = (long long)blockIdx.x * DW_WG_STRIPS + k; s < strips; s += (long long)gridDim.x * DW_WG_STRIPS) {
            const int w0 = (int)(s % strips_w) * 4;
            const long long R = s / strips_w;
            const int h = (int)(R % H);
            const int hi = h - 1 + rr;
            if (hi < 0 || hi >= H) continue;
            float d[4][V], in[6][V];
            const T* row = x + ((R - h + hi) * W) * (long long)C + c;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (w0 + j < W) ldv<V>(dy + ((R * W) + w0 + j) * (long long)C + c, d[j]);
                else {
#pragma unroll
                    for (int e = 0; e < V; ++e) d[j][e] = 0.f;
                }
            }
#pragma unroll
            for (int j = 0; j < 6; ++j) {
                const int wi = w0 - 1 + j;
                if (wi >= 0 && wi < W) {
                    ldv<V>(row + (long long)wi * C, in[j]);
                    if constexpr (XF) xr.apply(in[j]);
                } else {
#pragma unroll
                    for (int e = 0; e < V; ++e) in[j][e] = 0.f;
                }
            }
#pragma unroll
            for (int ss = 0; ss < 3; ++ss)
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int e = 0; e < V; ++e) acc[ss][e] = fmaf(in[j + ss][e], d[j][e], acc[ss][e]);
        }
    }
#pragma unroll
    for (int t = 0; t < 3; ++t)
#pragma unroll
        for (int e = 0; e < V; ++e) sh[t][slot][cvl * V + e] = acc[t][e];
    __syncthreads();
    for (int q = threadIdx.x; q < 9 * 8 * V; q += 256) {
        const int tap = q / (8 * V), cc = q % (8 * V), gq = tap / 3, t = tap - 3 * gq;
        const int gc = blockIdx.y * 8 * V + cc;
        if (gc < C) {
            float sum = 0.f;
#pragma unroll
            for (int kk = 0; kk < DW_WG_STRIPS; ++kk) sum += sh[t][3 * kk + gq][cc];
            partial[((long long)blockIdx.x * 9 + tap) * C + gc] = sum;
        }
    }
}

// dw[t][c] = sum over chunks and folded copies of partial[chunk][t][copy * C + c]; grid (ceil(C/32), G, 9)
__global__ void dw_wgrad_finalize_kernel(const float* __restrict__ partial, int chunks, int f, int C, int cols, float* __restrict__ dw,
                                         const FinScratch fin) {
    grid_dep_sync();
    const int c = blockIdx.x * FIN_X + threadIdx.x;
    double ss[1];
    if (!col_fold_sums<float, 1>(partial, (int)blockIdx.z, 9, chunks, f, C, cols, c, fin, ss)) return;
    if (threadIdx.y == 0 && c < C) dw[blockIdx.z * C + c] = (float)ss[0];
}

// The same sum when a channel has few partial sums (at most DW_FIN_SMALL): one block of 32 channels x 8 runs per tap
// instead of 1024-thread blocks per eight channels.  grid (ceil(C/32), 9), block (32, 8); the runs are added in order.
constexpr int DW_FIN_SMALL = 512;
__global__ void __launch_bounds__(256) dw_wgrad_finalize_small_kernel(const float* __restrict__ partial, int chunks, int f, int C, int cols,
                                                                      float* __restrict__ dw) {
    grid_dep_sync();
    __shared__ double sh[8][32];
    const int c = blockIdx.x * 32 + threadIdx.x, t = blockIdx.y, total = chunks * f;
    double a = 0.0;
    if (c < C) {
#pragma unroll 4
        for (int e = threadIdx.y; e < total; e += 8) {
            const int ch = e / f, k = e - ch * f;
            a += (double)partial[((long long)ch * 9 + t) * cols + k * C + c];
        }
    }
    sh[threadIdx.y][threadIdx.x] = a;
    __syncthreads();
    if (threadIdx.y == 0 && c < C) {
        double r = 0.0;
#pragma unroll
        for (int y = 0; y < 8; ++y) r += sh[y][threadIdx.x];
        dw[t * C + c] = (float)r;
    }
}

// ---- stride-1 depthwise 3x3 on column strips, marching down the rows ---------------------------------------------
// A thread owns four channels and a strip of four output columns and walks down RH rows of one image with the
// three input rows of its window (3 x 6 vectors) in registers: every step loads one new row, so an input vector
// is fetched (RH + 2) / RH * 1.5 times instead of 4.5 times, and a batch norm folded into the load (XF) is
// evaluated once per fetch.  Block: 8 channel vectors x 32 slots; a slot is (image, row chunk, strip), numbered
// row-major.  Per output the taps are added in the order of dw_strip_kernel, so both give the same bits.
template <typename T>
__device__ __forceinline__ void dw3_fetch_row(const T* __restrict__ img, int hi, int H, int W, int C, int w0, float (&r)[6][4]) {
#pragma unroll
    for (int j = 0; j < 6; ++j) {
        const int wi = w0 - 1 + j;
        if (hi >= 0 && hi < H && wi >= 0 && wi < W) ldv<4>(img + ((long long)hi * W + wi) * C, r[j]);
        else {
#pragma unroll
            for (int e = 0; e < 4; ++e) r[j][e] = 0.f;
        }
    }
}
// a fetched row becomes a window row: the batch norm of the tensor's producer, where one is folded in (padding stays zero)
template <typename T, bool XF>
__device__ __forceinline__ void dw3_take_row(const float (&raw)[6][4], int hi, int H, int W, int w0, float (&r)[6][4], const XfRegs<T, 4>& xr) {
#pragma unroll
    for (int j = 0; j < 6; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) r[j][e] = raw[j][e];
        if constexpr (XF) {
            const int wi = w0 - 1 + j;
            if (hi >= 0 && hi < H && wi >= 0 && wi < W) xr.apply(r[j]);
        }
    }
}
template <typename T, bool XF>
__device__ __forceinline__ void dw3_load_row(const T* __restrict__ img, int hi, int H, int W, int C, int w0, float (&r)[6][4], const XfRegs<T, 4>& xr) {
    float raw[6][4];
    dw3_fetch_row<T>(img, hi, H, W, C, w0, raw);
    dw3_take_row<T, XF>(raw, hi, H, W, w0, r, xr);
}

template <typename T, bool XF, bool STATS>
__global__ void __launch_bounds__(256, XF ? 1 : 2) dw3_fwd_rows_kernel(const T* __restrict__ x, const float* __restrict__ w, T* __restrict__ y, int N, int H, int W,
                                                              int C, int RH, int HC, double* __restrict__ stats, BnXform xf) {
    grid_dep_sync();
    __shared__ __align__(16) float wsm[9][32];
    __shared__ float shs[STATS ? 2 : 1][32][33];
    const int CV = C / 4, cvl = threadIdx.x & 7, slot = threadIdx.x >> 3, cv = blockIdx.y * 8 + cvl, c = cv * 4;
    for (int i = threadIdx.x; i < 9 * 32; i += 256) {
        const int tap = i >> 5, ch = blockIdx.y * 32 + (i & 31);
        wsm[tap][i & 31] = ch < C ? w[tap * C + ch] : 0.f;
    }
    __syncthreads();
    const int strips_w = (W + 3) >> 2;
    const long long total = (long long)N * HC * strips_w;
    float su[4] = {0.f, 0.f, 0.f, 0.f}, sq[4] = {0.f, 0.f, 0.f, 0.f};
    for (long long gs = (long long)blockIdx.x * 32 + slot; cv < CV && gs < total; gs += (long long)gridDim.x * 32) {
        const int sw = (int)(gs % strips_w);
        const long long t = gs / strips_w;
        const int hc = (int)(t % HC), n = (int)(t / HC);
        const int w0 = sw * 4, h0 = hc * RH, h1 = min(H, h0 + RH);
        XfRegs<T, 4> xr;
        if constexpr (XF) xr.load(xf, c);
        const T* img = x + (long long)n * H * W * C + c;
        T* out = y + (long long)n * H * W * C + c;
        float win[3][6][4], nxt[6][4];
        dw3_load_row<T, XF>(img, h0 - 1, H, W, C, w0, win[0], xr);
        dw3_load_row<T, XF>(img, h0, H, W, C, w0, win[1], xr);
        dw3_fetch_row<T>(img, h0 + 1, H, W, C, w0, nxt);
        for (int h = h0; h < h1; ++h) {
            dw3_take_row<T, XF>(nxt, h + 1, H, W, w0, win[2], xr);
            if (h + 1 < h1) dw3_fetch_row<T>(img, h + 2, H, W, C, w0, nxt);         // in flight while this row is computed
            float acc[4][4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[j][e] = 0.f;
#pragma unroll
            for (int r = 0; r < 3; ++r)
#pragma unroll
                for (int s = 0; s < 3; ++s) {
                    const float4 kk = *reinterpret_cast<const float4*>(&wsm[r * 3 + s][cvl * 4]);
                    const float k4[4] = {kk.x, kk.y, kk.z, kk.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j)
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[j][e] = fmaf(win[r][j + s][e], k4[e], acc[j][e]);
                }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (w0 + j < W) {
                    stv<4>(out + ((long long)h * W + w0 + j) * C, acc[j]);
                    if constexpr (STATS) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) { const float v = as_stored<T>(acc[j][e]); su[e] += v; sq[e] = fmaf(v, v, sq[e]); }
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < 6; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) { win[0][j][e] = win[1][j][e]; win[1][j][e] = win[2][j][e]; }
        }
    }
    if constexpr (STATS) {
#pragma unroll
        for (int e = 0; e < 4; ++e) { shs[0][slot][cvl * 4 + e] = su[e]; shs[1][slot][cvl * 4 + e] = sq[e]; }
        __syncthreads();
        if (threadIdx.x < 64) {
            const int a = threadIdx.x >> 5, ch = threadIdx.x & 31, gc = blockIdx.y * 32 + ch;
            if (gc < C) {
                double tsum = 0.0;
#pragma unroll
                for (int q = 0; q < 32; ++q) tsum += (double)shs[a][q][ch];
                stats[((long long)blockIdx.x * 2 + a) * C + gc] = tsum;
            }
        }
    }
}

// Data gradient and weight gradient of the same convolution in one pass over dy: with the 3 x 6 window of output
// gradients around its four pixels of a row in registers, a thread forms dx (the taps mirrored, added in the
// order of dw_strip_kernel<FLIP = 1>) and adds x[pixel] * dy[pixel + offset] to the nine weight-gradient sums of its
// four channels, which it carries down its rows.  At the end the 32 slots of a block are added in slot order:
// partial[blockIdx.x][9][C] (float), summed over blocks by the finalize kernels.  dx may be NULL (no input gradient).
// BST (with XF): x is the input of the batch norm that precedes this convolution, so dx is the gradient with respect to
// that batch norm's output: it is stored already masked by the batch norm's activation, and the block leaves the two sums
// of the batch norm's backward pass (of g and of g * xhat, g as stored) in bstats[blockIdx.x][2][C] -- the separate
// reduction pass over (dx, x) is not needed.
template <typename T, bool XF, bool BST>
__global__ void __launch_bounds__(256) dw3_bwd_rows_kernel(const T* __restrict__ x, const T* __restrict__ dy, const float* __restrict__ w,
                                                           const T* __restrict__ addend, T* __restrict__ dx, float* __restrict__ partial, int N, int H,
                                                           int W, int C, int RH, int HC, BnXform xf, const float* __restrict__ rstd,
                                                           double* __restrict__ bstats) {
    static_assert(!BST || XF, "the backward sums need the batch norm's input");
    grid_dep_sync();
    __shared__ __align__(16) float wsm[9][32];
    __shared__ float sh[3][32][33];
    float bs1[4] = {0.f, 0.f, 0.f, 0.f}, bs2[4] = {0.f, 0.f, 0.f, 0.f};
    const int CV = C / 4, cvl = threadIdx.x & 7, slot = threadIdx.x >> 3, cv = blockIdx.y * 8 + cvl, c = cv * 4;
    for (int i = threadIdx.x; i < 9 * 32; i += 256) {
        const int tap = i >> 5, ch = blockIdx.y * 32 + (i & 31);
        wsm[tap][i & 31] = ch < C ? w[tap * C + ch] : 0.f;
    }
    __syncthreads();
    const int strips_w = (W + 3) >> 2;
    const long long total = (long long)N * HC * strips_w;
    float dwa[9][4];
#pragma unroll
    for (int tap = 0; tap < 9; ++tap)
#pragma unroll
        for (int e = 0; e < 4; ++e) dwa[tap][e] = 0.f;
    for (long long gs = (long long)blockIdx.x * 32 + slot; cv < CV && gs < total; gs += (long long)gridDim.x * 32) {
        const int sw = (int)(gs % strips_w);
        const long long t = gs / strips_w;
        const int hc = (int)(t % HC), n = (int)(t / HC);
        const int w0 = sw * 4, h0 = hc * RH, h1 = min(H, h0 + RH);
        XfRegs<T, 4> xr, none;
        if constexpr (XF) xr.load(xf, c);
        float rs[4] = {0.f, 0.f, 0.f, 0.f};
        if constexpr (BST) ldtab<4>(rstd + c, rs);
        const long long ioff = (long long)n * H * W * C + c;
        const T* gimg = dy + ioff;
        float win[3][6][4];
        dw3_load_row<T, false>(gimg, h0 - 1, H, W, C, w0, win[0], none);
        dw3_load_row<T, false>(gimg, h0, H, W, C, w0, win[1], none);
        dw3_fetch_row<T>(gimg, h0 + 1, H, W, C, w0, win[2]);
        float xnext[4][4];
        auto fetch_x = [&](int h) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (w0 + j < W) ldv<4>(x + ioff + ((long long)h * W + w0 + j) * C, xnext[j]);
                else {
#pragma unroll
                    for (int e = 0; e < 4; ++e) xnext[j][e] = 0.f;
                }
            }
        };
        fetch_x(h0);
        for (int h = h0; h < h1; ++h) {
            float xv[4][4], acc[4][4], xh[BST ? 4 : 1][4];
            unsigned pass = 0u;                                  // bit 4 j + e: the activation lets the gradient through
#pragma unroll
            for (int j = 0; j < 4; ++j) {
#pragma unroll
                for (int e = 0; e < 4; ++e) { xv[j][e] = xnext[j][e]; acc[j][e] = 0.f; }
                if constexpr (BST) {
                    if (w0 + j < W) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float cen = xv[j][e] - xr.mu[e], z = fmaf(cen, xr.sc[e], xr.of[e]);
                            xh[j][e] = cen * rs[e];
                            if (z > xr.lo && z < xr.hi) pass |= 1u << (4 * j + e);
                            xv[j][e] = as_stored<T>(fminf(fmaxf(z, xr.lo), xr.hi));
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 4; ++e) xh[j][e] = 0.f;
                    }
                } else if constexpr (XF) { if (w0 + j < W) xr.apply(xv[j]); }
            }
            if (h + 1 < h1) fetch_x(h + 1);                      // lands while this row is computed
#pragma unroll
            for (int r = 0; r < 3; ++r)
#pragma unroll
                for (int s = 0; s < 3; ++s) {
                    const int tap = (2 - r) * 3 + (2 - s);
                    const float4 kk = *reinterpret_cast<const float4*>(&wsm[tap][cvl * 4]);
                    const float k4[4] = {kk.x, kk.y, kk.z, kk.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            acc[j][e] = fmaf(win[r][j + s][e], k4[e], acc[j][e]);
                            dwa[tap][e] = fmaf(xv[j][e], win[r][j + s][e], dwa[tap][e]);
                        }
                }
            // the window moves down one row; the row after it is fetched now and lands while the next x row is awaited
#pragma unroll
            for (int j = 0; j < 6; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) { win[0][j][e] = win[1][j][e]; win[1][j][e] = win[2][j][e]; }
            if (h + 1 < h1) dw3_fetch_row<T>(gimg, h + 2, H, W, C, w0, win[2]);
            if (dx) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (w0 + j < W) {
                        const long long o = ioff + ((long long)h * W + w0 + j) * C;
                        if (addend) {
                            float a[4];
                            ldv<4>(addend + o, a);
#pragma unroll
                            for (int e = 0; e < 4; ++e) acc[j][e] += a[e];
                        }
                        if constexpr (BST) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float gq = (pass >> (4 * j + e)) & 1u ? as_stored<T>(acc[j][e]) : 0.f;
                                acc[j][e] = gq;
                                bs1[e] += gq;
                                bs2[e] = fmaf(gq, xh[j][e], bs2[e]);
                            }
                        }
                        stv<4>(dx + o, acc[j]);
                    }
                }
            }
        }
    }
    if constexpr (BST) {
        // the two sums of every channel over the block's 32 slots, in slot order, as doubles
        __syncthreads();
#pragma unroll
        for (int e = 0; e < 4; ++e) { sh[0][slot][cvl * 4 + e] = bs1[e]; sh[1][slot][cvl * 4 + e] = bs2[e]; }
        __syncthreads();
        if (threadIdx.x < 64) {
            const int a = threadIdx.x >> 5, ch = threadIdx.x & 31, gc = blockIdx.y * 32 + ch;
            if (gc < C) {
                double tsum = 0.0;
#pragma unroll 8
                for (int q = 0; q < 32; ++q) tsum += (double)sh[a][q][ch];
                bstats[((long long)blockIdx.x * 2 + a) * C + gc] = tsum;
            }
        }
    }
    // the nine sums of every channel over the block's 32 slots, three taps at a time, in slot order
#pragma unroll
    for (int gq = 0; gq < 3; ++gq) {
        __syncthreads();
#pragma unroll
        for (int tq = 0; tq < 3; ++tq)
#pragma unroll
            for (int e = 0; e < 4; ++e) sh[tq][slot][cvl * 4 + e] = dwa[gq * 3 + tq][e];
        __syncthreads();
        if (threadIdx.x < 96) {
            const int tq = threadIdx.x >> 5, ch = threadIdx.x & 31, gc = blockIdx.y * 32 + ch;
            if (gc < C) {
                float sum = 0.f;
#pragma unroll 8
                for (int q = 0; q < 32; ++q) sum += sh[tq][q][ch];
                partial[((long long)blockIdx.x * 9 + gq * 3 + tq) * C + gc] = sum;
            }
        }
    }
}

// ---- stride-2 depthwise 3x3 (pad 1) on column strips, marching down the output rows ------------------------------
// A thread owns four channels and two neighbouring output columns (input columns 2 wo0 - 1 .. 2 wo0 + 3) and walks
// down RH output rows of one image.  Output row ho reads input rows 2 ho - 1, 2 ho, 2 ho + 1; the thread takes the
// input rows in order, one pair per step with the next pair in flight, and carries the contribution of row 2 ho + 1
// to output row ho + 1 (filter row 0) in registers, so every input row is fetched once per strip.  Block and slot
// numbering as in the stride-1 kernels above (a slot is (image, row chunk, strip of two output columns)).
template <typename T>
__device__ __forceinline__ void dws2_fetch_row(const T* __restrict__ img, int hi, int H, int W, int C, int wi0, float (&r)[5][4]) {
#pragma unroll
    for (int j = 0; j < 5; ++j) {
        const int wi = wi0 + j;
        if (hi >= 0 && hi < H && wi >= 0 && wi < W) ldv<4>(img + ((long long)hi * W + wi) * C, r[j]);
        else {
#pragma unroll
            for (int e = 0; e < 4; ++e) r[j][e] = 0.f;
        }
    }
}
template <typename T, bool XF>
__device__ __forceinline__ void dws2_take_row(const float (&raw)[5][4], int hi, int H, int W, int wi0, float (&r)[5][4], const XfRegs<T, 4>& xr) {
#pragma unroll
    for (int j = 0; j < 5; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) r[j][e] = raw[j][e];
        if constexpr (XF) {
            const int wi = wi0 + j;
            if (hi >= 0 && hi < H && wi >= 0 && wi < W) xr.apply(r[j]);
        }
    }
}
// acc[j] += sum over the three taps of filter row `fr` of z[2 j + s] * w[fr][s]
__device__ __forceinline__ void dws2_row_taps(const float (&z)[5][4], const float (*wsm)[32], int fr, int cvl, float (&acc)[2][4]) {
#pragma unroll
    for (int s = 0; s < 3; ++s) {
        const float4 kk = *reinterpret_cast<const float4*>(&wsm[fr * 3 + s][cvl * 4]);
        const float k4[4] = {kk.x, kk.y, kk.z, kk.w};
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[j][e] = fmaf(z[2 * j + s][e], k4[e], acc[j][e]);
    }
}

template <typename T, bool XF, bool STATS>
__global__ void __launch_bounds__(256, 2) dw3s2_fwd_rows_kernel(const T* __restrict__ x, const float* __restrict__ w, T* __restrict__ y, int N, int H, int W,
                                                                int C, int Ho, int Wo, int RH, int HC, double* __restrict__ stats, BnXform xf) {
    grid_dep_sync();
    __shared__ __align__(16) float wsm[9][32];
    __shared__ float shs[STATS ? 2 : 1][32][33];
    const int CV = C / 4, cvl = threadIdx.x & 7, slot = threadIdx.x >> 3, cv = blockIdx.y * 8 + cvl, c = cv * 4;
    for (int i = threadIdx.x; i < 9 * 32; i += 256) {
        const int tap = i >> 5, ch = blockIdx.y * 32 + (i & 31);
        wsm[tap][i & 31] = ch < C ? w[tap * C + ch] : 0.f;
    }
    __syncthreads();
    const int strips_w = (Wo + 1) >> 1;
    const long long total = (long long)N * HC * strips_w;
    float su[4] = {0.f, 0.f, 0.f, 0.f}, sq[4] = {0.f, 0.f, 0.f, 0.f};
    for (long long gs = (long long)blockIdx.x * 32 + slot; cv < CV && gs < total; gs += (long long)gridDim.x * 32) {
        const int sw = (int)(gs % strips_w);
        const long long t = gs / strips_w;
        const int hc = (int)(t % HC), n = (int)(t / HC);
        const int wo0 = sw * 2, wi0 = 2 * wo0 - 1, h0 = hc * RH, h1 = min(Ho, h0 + RH);
        XfRegs<T, 4> xr;
        if constexpr (XF) xr.load(xf, c);
        const T* img = x + (long long)n * H * W * C + c;
        T* out = y + (long long)n * Ho * Wo * C + c;
        float ra[5][4], rb[5][4], z[5][4], acc[2][4], accn[2][4];
        dws2_fetch_row<T>(img, 2 * h0 - 1, H, W, C, wi0, rb);
        dws2_fetch_row<T>(img, 2 * h0, H, W, C, wi0, ra);
        dws2_take_row<T, XF>(rb, 2 * h0 - 1, H, W, wi0, z, xr);
        dws2_fetch_row<T>(img, 2 * h0 + 1, H, W, C, wi0, rb);
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) accn[j][e] = 0.f;
        dws2_row_taps(z, wsm, 0, cvl, accn);
        for (int ho = h0; ho < h1; ++ho) {
            const bool more = ho + 1 < h1;
#pragma unroll
            for (int j = 0; j < 2; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) { acc[j][e] = accn[j][e]; accn[j][e] = 0.f; }
            dws2_take_row<T, XF>(ra, 2 * ho, H, W, wi0, z, xr);
            if (more) dws2_fetch_row<T>(img, 2 * ho + 2, H, W, C, wi0, ra);            // in flight while these rows are computed
            dws2_row_taps(z, wsm, 1, cvl, acc);
            dws2_take_row<T, XF>(rb, 2 * ho + 1, H, W, wi0, z, xr);
            if (more) dws2_fetch_row<T>(img, 2 * ho + 3, H, W, C, wi0, rb);
            dws2_row_taps(z, wsm, 2, cvl, acc);
            dws2_row_taps(z, wsm, 0, cvl, accn);
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                if (wo0 + j < Wo) {
                    stv<4>(out + ((long long)ho * Wo + wo0 + j) * C, acc[j]);
                    if constexpr (STATS) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) { const float v = as_stored<T>(acc[j][e]); su[e] += v; sq[e] = fmaf(v, v, sq[e]); }
                    }
                }
            }
        }
    }
    if constexpr (STATS) {
#pragma unroll
        for (int e = 0; e < 4; ++e) { shs[0][slot][cvl * 4 + e] = su[e]; shs[1][slot][cvl * 4 + e] = sq[e]; }
        __syncthreads();
        if (threadIdx.x < 64) {
            const int a = threadIdx.x >> 5, ch = threadIdx.x & 31, gc = blockIdx.y * 32 + ch;
            if (gc < C) {
                double tsum = 0.0;
#pragma unroll
                for (int q = 0; q < 32; ++q) tsum += (double)shs[a][q][ch];
                stats[((long long)blockIdx.x * 2 + a) * C + gc] = tsum;
            }
        }
    }
}

// Backward of the same convolution in one pass.  For output row ho the thread holds dy of rows ho and ho + 1 (columns
// wo0 .. wo0 + 2) and takes input rows 2 ho (even) and 2 ho + 1 (odd), columns 2 wo0 - 1 .. 2 wo0 + 3:
//   weight gradient: row 2 ho meets filter row 1 with dy[ho]; row 2 ho + 1 meets filter row 2 with dy[ho] and filter
//   row 0 with dy[ho + 1] -- so no input row is carried from step to step;
//   data gradient of its four input columns 2 wo0 .. 2 wo0 + 3 in both rows: an even row or column receives the middle
//   tap of one output, an odd one the two outer taps of two outputs.
// partial[blockIdx.x][9][C], bstats[blockIdx.x][2][C] and the meaning of XF / BST are those of dw3_bwd_rows_kernel.
template <typename T>
__device__ __forceinline__ void dws2_fetch_dy(const T* __restrict__ gimg, int ho, int Ho, int Wo, int C, int wo0, float (&r)[3][4]) {
#pragma unroll
    for (int j = 0; j < 3; ++j) {
        if (ho < Ho && wo0 + j < Wo) ldv<4>(gimg + ((long long)ho * Wo + wo0 + j) * C, r[j]);
        else {
#pragma unroll
            for (int e = 0; e < 4; ++e) r[j][e] = 0.f;
        }
    }
}

template <typename T, bool XF, bool BST>
__global__ void __launch_bounds__(256) dw3s2_bwd_rows_kernel(const T* __restrict__ x, const T* __restrict__ dy, const float* __restrict__ w,
                                                             const T* __restrict__ addend, T* __restrict__ dx, float* __restrict__ partial, int N, int H,
                                                             int W, int C, int Ho, int Wo, int RH, int HC, BnXform xf, const float* __restrict__ rstd,
                                                             double* __restrict__ bstats) {
    static_assert(!BST || XF, "the backward sums need the batch norm's input");
    grid_dep_sync();
    __shared__ __align__(16) float wsm[9][32];
    __shared__ float sh[3][32][33];
    float bs1[4] = {0.f, 0.f, 0.f, 0.f}, bs2[4] = {0.f, 0.f, 0.f, 0.f};
    const int CV = C / 4, cvl = threadIdx.x & 7, slot = threadIdx.x >> 3, cv = blockIdx.y * 8 + cvl, c = cv * 4;
    for (int i = threadIdx.x; i < 9 * 32; i += 256) {
        const int tap = i >> 5, ch = blockIdx.y * 32 + (i & 31);
        wsm[tap][i & 31] = ch < C ? w[tap * C + ch] : 0.f;
    }
    __syncthreads();
    const int strips_w = (Wo + 1) >> 1;
    const long long total = (long long)N * HC * strips_w;
    float dwa[9][4];
#pragma unroll
    for (int tap = 0; tap < 9; ++tap)
#pragma unroll
        for (int e = 0; e < 4; ++e) dwa[tap][e] = 0.f;
    for (long long gs = (long long)blockIdx.x * 32 + slot; cv < CV && gs < total; gs += (long long)gridDim.x * 32) {
        const int sw = (int)(gs % strips_w);
        const long long t = gs / strips_w;
        const int hc = (int)(t % HC), n = (int)(t / HC);
        const int wo0 = sw * 2, wi0 = 2 * wo0 - 1, h0 = hc * RH, h1 = min(Ho, h0 + RH);
        XfRegs<T, 4> xr;
        if constexpr (XF) xr.load(xf, c);
        float rs[4] = {0.f, 0.f, 0.f, 0.f};
        if constexpr (BST) ldtab<4>(rstd + c, rs);
        const long long ioff = (long long)n * H * W * C + c;
        const T* ximg = x + ioff;
        const T* gimg = dy + (long long)n * Ho * Wo * C + c;
        float cur[3][4], nxt[3][4], ra[5][4], rb[5][4];
        dws2_fetch_dy<T>(gimg, h0, Ho, Wo, C, wo0, cur);
        dws2_fetch_dy<T>(gimg, h0 + 1, Ho, Wo, C, wo0, nxt);
        dws2_fetch_row<T>(ximg, 2 * h0, H, W, C, wi0, ra);
        dws2_fetch_row<T>(ximg, 2 * h0 + 1, H, W, C, wi0, rb);
        for (int ho = h0; ho < h1; ++ho) {
            const bool more = ho + 1 < h1;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int hi = 2 * ho + half;
                float z[5][4], xh[BST ? 4 : 1][4], acc[4][4];
                unsigned pass = 0u;                              // bit 4 q + e: the activation lets the gradient of column 2 wo0 + q through
#pragma unroll
                for (int j = 0; j < 5; ++j) {
                    const int wi = wi0 + j;
                    const bool in = hi < H && wi >= 0 && wi < W;
#pragma unroll
                    for (int e = 0; e < 4; ++e) z[j][e] = half ? rb[j][e] : ra[j][e];
                    if constexpr (BST) {
                        if (in) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float cen = z[j][e] - xr.mu[e], v = fmaf(cen, xr.sc[e], xr.of[e]);
                                if (j > 0) {
                                    xh[j > 0 ? j - 1 : 0][e] = cen * rs[e];
                                    if (v > xr.lo && v < xr.hi) pass |= 1u << (4 * (j > 0 ? j - 1 : 0) + e);
                                }
                                z[j][e] = as_stored<T>(fminf(fmaxf(v, xr.lo), xr.hi));
                            }
                        } else if (j > 0) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) xh[j > 0 ? j - 1 : 0][e] = 0.f;
                        }
                    } else if constexpr (XF) { if (in) xr.apply(z[j]); }
                }
                // the row's buffer is free: the row two below lands while this one is used
                if (more) { if (half) dws2_fetch_row<T>(ximg, hi + 2, H, W, C, wi0, rb); else dws2_fetch_row<T>(ximg, hi + 2, H, W, C, wi0, ra); }
                // weight gradient
#pragma unroll
                for (int s = 0; s < 3; ++s)
#pragma unroll
                    for (int j = 0; j < 2; ++j)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            if (half) {
                                dwa[6 + s][e] = fmaf(z[2 * j + s][e], cur[j][e], dwa[6 + s][e]);
                                dwa[s][e] = fmaf(z[2 * j + s][e], nxt[j][e], dwa[s][e]);
                            } else dwa[3 + s][e] = fmaf(z[2 * j + s][e], cur[j][e], dwa[3 + s][e]);
                        }
                if (dx && hi < H) {
                    // data gradient of columns 2 wo0 + q, q = 0 .. 3
                    auto tap4 = [&](int tap, float (&k4)[4]) {
                        const float4 kk = *reinterpret_cast<const float4*>(&wsm[tap][cvl * 4]);
                        k4[0] = kk.x; k4[1] = kk.y; k4[2] = kk.z; k4[3] = kk.w;
                    };
                    if (!half) {
                        float k0[4], k1[4], k2[4];
                        tap4(3, k0); tap4(4, k1); tap4(5, k2);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            acc[0][e] = k1[e] * cur[0][e];
                            acc[1][e] = fmaf(k2[e], cur[0][e], k0[e] * cur[1][e]);
                            acc[2][e] = k1[e] * cur[1][e];
                            acc[3][e] = fmaf(k2[e], cur[1][e], k0[e] * cur[2][e]);
                        }
                    } else {
                        float t0[4], t1[4], t2[4], b0[4], b1[4], b2[4];
                        tap4(0, t0); tap4(1, t1); tap4(2, t2); tap4(6, b0); tap4(7, b1); tap4(8, b2);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            acc[0][e] = fmaf(b1[e], cur[0][e], t1[e] * nxt[0][e]);
                            acc[1][e] = fmaf(b2[e], cur[0][e], fmaf(b0[e], cur[1][e], fmaf(t2[e], nxt[0][e], t0[e] * nxt[1][e])));
                            acc[2][e] = fmaf(b1[e], cur[1][e], t1[e] * nxt[1][e]);
                            acc[3][e] = fmaf(b2[e], cur[1][e], fmaf(b0[e], cur[2][e], fmaf(t2[e], nxt[1][e], t0[e] * nxt[2][e])));
                        }
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int wi = 2 * wo0 + q;
                        if (wi < W) {
                            const long long o = ioff + ((long long)hi * W + wi) * C;
                            if (addend) {
                                float a[4];
                                ldv<4>(addend + o, a);
#pragma unroll
                                for (int e = 0; e < 4; ++e) acc[q][e] += a[e];
                            }
                            if constexpr (BST) {
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const float gq = (pass >> (4 * q + e)) & 1u ? as_stored<T>(acc[q][e]) : 0.f;
                                    acc[q][e] = gq;
                                    bs1[e] += gq;
                                    bs2[e] = fmaf(gq, xh[q][e], bs2[e]);
                                }
                            }
                            stv<4>(dx + o, acc[q]);
                        }
                    }
                }
            }
            // dy moves down one output row
#pragma unroll
            for (int j = 0; j < 3; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) cur[j][e] = nxt[j][e];
            if (more) dws2_fetch_dy<T>(gimg, ho + 2, Ho, Wo, C, wo0, nxt);
        }
    }
    if constexpr (BST) {
        __syncthreads();
#pragma unroll
        for (int e = 0; e < 4; ++e) { sh[0][slot][cvl * 4 + e] = bs1[e]; sh[1][slot][cvl * 4 + e] = bs2[e]; }
        __syncthreads();
        if (threadIdx.x < 64) {
            const int a = threadIdx.x >> 5, ch = threadIdx.x & 31, gc = blockIdx.y * 32 + ch;
            if (gc < C) {
                double tsum = 0.0;
#pragma unroll 8
                for (int q = 0; q < 32; ++q) tsum += (double)sh[a][q][ch];
                bstats[((long long)blockIdx.x * 2 + a) * C + gc] = tsum;
            }
        }
    }
#pragma unroll
    for (int gq = 0; gq < 3; ++gq) {
        __syncthreads();
#pragma unroll
        for (int tq = 0; tq < 3; ++tq)
#pragma unroll
            for (int e = 0; e < 4; ++e) sh[tq][slot][cvl * 4 + e] = dwa[gq * 3 + tq][e];
        __syncthreads();
        if (threadIdx.x < 96) {
            const int tq = threadIdx.x >> 5, ch = threadIdx.x & 31, gc = blockIdx.y * 32 + ch;
            if (gc < C) {
                float sum = 0.f;
#pragma unroll 8
                for (int q = 0; q < 32; ++q) sum += sh[tq][q][ch];
                partial[((long long)blockIdx.x * 9 + gq * 3 + tq) * C + gc] = sum;
            }
        }
    }
}

// ---- pooling --------------------------------------------------------------------------------------
template <typename T, int V>
__global__ void __launch_bounds__(256) maxpool_fwd_kernel(const T* __restrict__ x, T* __restrict__ y, int H, int W, int C, long long total) {
    grid_dep_sync();
    const int CV = C / V, Ho = H / 2, Wo = W / 2;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(i % CV) * V;
        long long pix = i / CV;
        const int wo = (int)(pix % Wo); pix /= Wo;
        const int ho = (int)(pix % Ho);
        const int n = (int)(pix / Ho);
        float m[V];
        ldv<V>(x + ((long long)(n * H + 2 * ho) * W + 2 * wo) * C + c, m);
#pragma unroll
        for (int q = 1; q < 4; ++q) {
            float v[V];
            ldv<V>(x + ((long long)(n * H + 2 * ho + (q >> 1)) * W + 2 * wo + (q & 1)) * C + c, v);
#pragma unroll
            for (int e = 0; e < V; ++e) m[e] = v[e] > m[e] ? v[e] : m[e];
        }
        stv<V>(y + i * V, m);
    }
}

// one thread per output pixel / channel vector writes its four inputs: the gradient goes to the first
// maximum in row-major window order, zero elsewhere (rows/columns beyond 2*floor(H/2) get zero too)
template <typename T, int V>
__global__ void __launch_bounds__(256) maxpool_bwd_kernel(const T* __restrict__ dy, const T* __restrict__ x, T* __restrict__ dx, int H, int W, int C, long long total) {
    grid_dep_sync();
    const int CV = C / V, Ho = H / 2, Wo = W / 2;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(i % CV) * V;
        long long pix = i / CV;
        const int wo = (int)(pix % Wo); pix /= Wo;
        const int ho = (int)(pix % Ho);
        const int n = (int)(pix / Ho);
        float v[4][V], d[V];
        int arg[V];
        ldv<V>(dy + i * V, d);
#pragma unroll
        for (int q = 0; q < 4; ++q) ldv<V>(x + ((long long)(n * H + 2 * ho + (q >> 1)) * W + 2 * wo + (q & 1)) * C + c, v[q]);
#pragma unroll
        for (int e = 0; e < V; ++e) {
            arg[e] = 0;
            float m = v[0][e];
#pragma unroll
            for (int q = 1; q < 4; ++q) if (v[q][e] > m) { m = v[q][e]; arg[e] = q; }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float o[V];
#pragma unroll
            for (int e = 0; e < V; ++e) o[e] = arg[e] == q ? d[e] : 0.f;
            stv<V>(dx + ((long long)(n * H + 2 * ho + (q >> 1)) * W + 2 * wo + (q & 1)) * C + c, o);
        }
    }
}

template <typename T, int V>
__global__ void __launch_bounds__(256) gap_fwd_kernel(const T* __restrict__ x, T* __restrict__ y, int HW, int C, long long total) {
    grid_dep_sync();
    const int CV = C / V;
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int c = (int)(i % CV) * V;
    const long long n = i / CV;
    float s[V];
#pragma unroll
    for (int e = 0; e < V; ++e) s[e] = 0.f;
    // eight positions per trip: their loads are issued together, the additions keep the order of the positions
    int p = 0;
    for (; p + 8 <= HW; p += 8) {
        float v[8][V];
#pragma unroll
        for (int u = 0; u < 8; ++u) ldv<V>(x + (n * HW + p + u) * C + c, v[u]);
#pragma unroll
        for (int u = 0; u < 8; ++u)
#pragma unroll
            for (int e = 0; e < V; ++e) s[e] += v[u][e];
    }
    for (; p < HW; ++p) {
        float v[V];
        ldv<V>(x + (n * HW + p) * C + c, v);
#pragma unroll
        for (int e = 0; e < V; ++e) s[e] += v[e];
    }
    const float inv = 1.f / (float)HW;
#pragma unroll
    for (int e = 0; e < V; ++e) s[e] *= inv;
    stv<V>(y + i * V, s);
}

template <typename T, int V>
__global__ void __launch_bounds__(256) gap_bwd_kernel(const T* __restrict__ dy, T* __restrict__ dx, int HW, int C, long long total) {
    grid_dep_sync();
    const int CV = C / V;
    const float inv = 1.f / (float)HW;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int cv = (int)(i % CV);
        const long long n = i / CV / HW;
        float v[V];
        ldv<V>(dy + (n * CV + cv) * V, v);
#pragma unroll
        for (int e = 0; e < V; ++e) v[e] *= inv;
        stv<V>(dx + i * V, v);
    }
}

// ---- softmax cross-entropy: one block per sample ---------------------------------------------------
__device__ __forceinline__ float block_reduce(float v, bool is_max, float* sh) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { const float u = __shfl_xor_sync(0xffffffffu, v, o); v = is_max ? fmaxf(v, u) : v + u; }
    __syncthreads();
    if (lane == 0) sh[wid] = v;
    __syncthreads();
    float r = sh[0];
    for (int i = 1; i < nw; ++i) r = is_max ? fmaxf(r, sh[i]) : r + sh[i];
    return r;
}

__global__ void __launch_bounds__(128) softmax_ce_kernel(const float* __restrict__ logits, const int32_t* __restrict__ labels, int N, int K,
                                                         float* __restrict__ per_sample, float* __restrict__ dlogits) {
    grid_dep_sync();
    __shared__ float sh[4];
    const int n = blockIdx.x;
    const float* z = logits + (long long)n * K;
    float mx = -FLT_MAX;
    for (int k = threadIdx.x; k < K; k += blockDim.x) mx = fmaxf(mx, z[k]);
    mx = block_reduce(mx, true, sh);
    float se = 0.f;
    for (int k = threadIdx.x; k < K; k += blockDim.x) se += expf(z[k] - mx);
    se = block_reduce(se, false, sh);
    int lab = labels[n];
    lab = lab < 0 ? 0 : (lab >= K ? K - 1 : lab);
    const float lse = logf(se);
    const float invn = 1.f / (float)N;
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        const float p = expf(z[k] - mx - lse);
        dlogits[(long long)n * K + k] = (p - (k == lab ? 1.f : 0.f)) * invn;
    }
    if (threadIdx.x == 0) per_sample[n] = -(z[lab] - mx - lse);
}

__global__ void loss_mean_kernel(const float* __restrict__ per_sample, int N, float* loss) {
    grid_dep_sync();
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        double s = 0.0;
        for (int i = 0; i < N; ++i) s += (double)per_sample[i];
        *loss = (float)(s / (double)N);
    }
}

// ---- SGD ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void sgd_one(float* w, const float* g, float* m, long long i, float lr, float mu, float wd, int first, __nv_bfloat16* shadow,
                                        float* lo, float* snap_dev, float* snap_host) {
    float wv = w[i], gv = fmaf(wd, wv, g[i]);
    if (m) {
        if (!first) gv = fmaf(mu, m[i], gv);
        m[i] = gv;
    }
    wv = fmaf(-lr, gv, wv);
    w[i] = wv;
    if (lo) lo[i] = wv - __uint_as_float(__float_as_uint(wv) & 0xffffe000u);
    if (snap_dev) snap_dev[i] = wv;
    if (snap_host) snap_host[i] = wv;
    if (shadow) shadow[i] = __float2bfloat16_rn(wv);
}

// nvec vectors of V parameters, then `tail` (< V) single parameters
template <int V>
__global__ void __launch_bounds__(256) sgd_kernel(float* __restrict__ w, const float* __restrict__ g, float* __restrict__ m, long long nvec, int tail, float lr,
                                                  float mu, float wd, int first, __nv_bfloat16* __restrict__ shadow, float* __restrict__ lo,
                                                  float* __restrict__ snap_dev, float* __restrict__ snap_host) {
    grid_dep_sync();
    if (blockIdx.x == 0 && (int)threadIdx.x < tail) sgd_one(w, g, m, nvec * V + threadIdx.x, lr, mu, wd, first, shadow, lo, snap_dev, snap_host);
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += (long long)gridDim.x * blockDim.x) {
        float wv[V], gv[V], mv[V];
        ldplain<V>(w + i * V, wv);           // w and m are written below: plain loads, not the read-only path
        ldv<V>(g + i * V, gv);
#pragma unroll
        for (int e = 0; e < V; ++e) gv[e] = fmaf(wd, wv[e], gv[e]);
        if (m) {
            if (!first) {
                ldplain<V>(m + i * V, mv);
#pragma unroll
                for (int e = 0; e < V; ++e) gv[e] = fmaf(mu, mv[e], gv[e]);
            }
            stv<V>(m + i * V, gv);
        }
#pragma unroll
        for (int e = 0; e < V; ++e) wv[e] = fmaf(-lr, gv[e], wv[e]);
        stv<V>(w + i * V, wv);
        if (lo) {
            float lv[V];
#pragma unroll
            for (int e = 0; e < V; ++e) lv[e] = wv[e] - __uint_as_float(__float_as_uint(wv[e]) & 0xffffe000u);
            stv<V>(lo + i * V, lv);
        }
        if (snap_dev) stv<V>(snap_dev + i * V, wv);
        if (snap_host) stv<V>(snap_host + i * V, wv);
        if (shadow) {
#pragma unroll
            for (int e = 0; e < V; ++e) shadow[i * V + e] = __float2bfloat16_rn(wv[e]);
        }
    }
}

__global__ void __launch_bounds__(256) mean_f32_kernel(MeanSources src, float* __restrict__ dst, long long count) {
    grid_dep_sync();
    const float inv = 1.f / (float)src.n;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (long long)gridDim.x * blockDim.x) {
        float a = src.p[0][i];
        for (int k = 1; k < src.n; ++k) a += src.p[k][i];
        dst[i] = a * inv;
    }
}

__global__ void f32_to_bf16_kernel(const float* __restrict__ s, __nv_bfloat16* __restrict__ d, long long n) {
    grid_dep_sync();
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        d[i] = __float2bfloat16_rn(s[i]);
}

__global__ void bf16_to_f32_kernel(const __nv_bfloat16* __restrict__ s, float* __restrict__ d, long long n) {
    grid_dep_sync();
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        d[i] = __bfloat162float(s[i]);
}

__global__ void tf32_lo_kernel(const float* __restrict__ w, float* __restrict__ lo, long long n) {
    grid_dep_sync();
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const float v = w[i];
        lo[i] = v - __uint_as_float(__float_as_uint(v) & 0xffffe000u);
    }
}

// One block per 32 x 32 tile of one of the matrices of the table: wt[n][k] = w[k][n], wtl[n][k] = its lo part.
__global__ void transpose_split_f32_kernel(const TransposeEntryDev* __restrict__ table, int n, int tile_base, const float* __restrict__ w,
                                           float* __restrict__ wt, float* __restrict__ wtl) {
    grid_dep_sync();
    __shared__ float tile[32][33];
    __shared__ int first_tile[256];
    const int t = tile_base + blockIdx.x;
    const int tid = threadIdx.y * 32 + threadIdx.x;
    int e = 0;
    if (n <= 256) {                     // the entries' first tiles, fetched by all threads at once instead of one after the other
        if (tid < n) first_tile[tid] = table[tid].tile0;
        __syncthreads();
        while (e + 1 < n && first_tile[e + 1] <= t) ++e;
    } else {
        while (e + 1 < n && table[e + 1].tile0 <= t) ++e;
    }
    const TransposeEntryDev en = table[e];
    const int local = t - en.tile0, tn = (en.N + 31) / 32;
    const int k0 = (local / tn) * 32, n0 = (local % tn) * 32;
    const float* src = w + en.w_off;
    for (int r = threadIdx.y; r < 32; r += 8) {
        const int k = k0 + r, c = n0 + threadIdx.x;
        tile[r][threadIdx.x] = (k < en.K && c < en.N) ? src[(long long)k * en.N + c] : 0.f;
    }
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += 8) {
        const int c = n0 + r, k = k0 + threadIdx.x;
        if (c < en.N && k < en.K) {
            const float v = tile[threadIdx.x][r];
            wt[en.w_off + (long long)c * en.K + k] = v;
            wtl[en.w_off + (long long)c * en.K + k] = v - __uint_as_float(__float_as_uint(v) & 0xffffe000u);
        }
    }
}

// The bf16 models' counterpart: wt[tap][n][k] = bf16(w[tap][k][n]) for every matrix of the table in one launch (an entry's
// `taps` matrices of K x N lie one after the other: 1 for a 1x1 convolution, 9 for a 3x3 one).
__global__ void transpose_bf16_batched_kernel(const TransposeEntryDev* __restrict__ table, int n, int tile_base, const float* __restrict__ w,
                                              __nv_bfloat16* __restrict__ wt) {
    grid_dep_sync();
    __shared__ float tile[32][33];
    __shared__ int first_tile[256];
    const int t = tile_base + blockIdx.x;
    const int tid = threadIdx.y * 32 + threadIdx.x;
    int e = 0;
    if (n <= 256) {
        if (tid < n) first_tile[tid] = table[tid].tile0;
        __syncthreads();
        while (e + 1 < n && first_tile[e + 1] <= t) ++e;
    } else {
        while (e + 1 < n && table[e + 1].tile0 <= t) ++e;
    }
    const TransposeEntryDev en = table[e];
    const int tn = (en.N + 31) / 32, per_tap = ((en.K + 31) / 32) * tn;
    const int local = t - en.tile0, tap = local / per_tap, in_tap = local - tap * per_tap;
    const int k0 = (in_tap / tn) * 32, n0 = (in_tap % tn) * 32;
    const long long base = en.w_off + (long long)tap * en.K * en.N;
    for (int r = threadIdx.y; r < 32; r += 8) {
        const int k = k0 + r, c = n0 + threadIdx.x;
        tile[r][threadIdx.x] = (k < en.K && c < en.N) ? w[base + (long long)k * en.N + c] : 0.f;
    }
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += 8) {
        const int c = n0 + r, k = k0 + threadIdx.x;
        if (c < en.N && k < en.K) wt[base + (long long)c * en.K + k] = __float2bfloat16_rn(tile[threadIdx.x][r]);
    }
}

template <typename T> inline bool can_vec(int C, const void* a, const void* b = nullptr, const void* c = nullptr, const void* d = nullptr) {
    return C % VecOf<T>::N == 0 && aligned16(a) && aligned16(b) && aligned16(c) && aligned16(d);
}

}  // namespace

// ---- host side ---------------------------------------------------------------------------------------------
FoldPlan make_fold(long long M, int C, int elem_bytes) {
    FoldPlan fp;
    const int V = 16 / elem_bytes;
    fp.vec = (C % V == 0) ? V : 1;
    fp.f = 1;
    if (fp.vec > 1) {
        const int tile = 32 * V;
        for (int f = 1; f <= 64; f *= 2)
            if (((long long)C * f) % tile == 0 && M % f == 0) { fp.f = f; break; }
    }
    fp.cols = C * fp.f;
    fp.rows = (int)(M / fp.f);
    const int coltiles = (fp.cols + 32 * fp.vec - 1) / (32 * fp.vec);
    // blocks per SM: the float kernels with the most registers (bn_bwd_apply, 80) hold three blocks per SM, so a grid of
    // four per SM runs a third of a second wave (config 2: 3.30 -> 3.27 ms per step with three); the bf16 kernels, which
    // move half the bytes per thread, measured better with four (config 3: 5.06 against 5.09 ms)
    const long long per_sm = elem_bytes == 4 ? 3 : 4;
    long long chunks = (per_sm * sm_count() + coltiles - 1) / coltiles;
    const long long maxc = (fp.rows + 15) / 16;
    if (chunks > maxc) chunks = maxc;
    if (chunks < 1) chunks = 1;
    // The reducing kernels merge the folded copies that fall inside one column tile.
    fp.fused = 0; fp.copies_fwd = fp.copies_bwd = 1;
    if (fp.vec > 1) {
        auto copies_in = [&](int tile) { return (tile % C == 0) ? std::min(fp.f, tile / C) : 1; };
        fp.copies_fwd = copies_in(32 * fp.vec); fp.copies_bwd = copies_in(128);
        fp.fused = 1;
    }
    const int rpc = (int)((fp.rows + chunks - 1) / chunks);
    fp.chunks = (fp.rows + rpc - 1) / rpc;
    return fp;
}

// up to this many partial sums per channel the second pass runs in blocks of FIN_X x FIN_Y_SMALL threads (one slice)
constexpr int FIN_SMALL_ENTRIES = 8 * FIN_Y_SMALL;
static inline int fin_slices_ps(const PartialSums& ps) {
    const int g = ps.entries / (4 * FIN_Y);
    return g < 1 ? 1 : (g > FIN_GMAX ? FIN_GMAX : g);
}

size_t fold_partial_doubles(const FoldPlan& fp) { return (size_t)fp.chunks * 2 * fp.cols; }

size_t fin_part_doubles(int C, int extra) { return (size_t)((C + FIN_X - 1) / FIN_X) * extra * FIN_GMAX * 2 * FIN_X; }
size_t fin_counter_count(int C, int extra) { return (size_t)((C + FIN_X - 1) / FIN_X) * extra; }
static inline int fin_slices(const FoldPlan& fp) {
    const int g = fp.chunks * fp.f / (4 * FIN_Y);
    return g < 1 ? 1 : (g > FIN_GMAX ? FIN_GMAX : g);
}

static inline int fold_rpc(const FoldPlan& fp) { return (fp.rows + fp.chunks - 1) / fp.chunks; }
static inline dim3 fold_grid(const FoldPlan& fp) { return dim3((fp.cols + 32 * fp.vec - 1) / (32 * fp.vec), fp.chunks); }
// the same row chunks walked with w columns per thread (w divides fp.vec)
static inline dim3 fold_grid_w(const FoldPlan& fp, int w) { return dim3((fp.cols + 32 * w - 1) / (32 * w), fp.chunks); }

size_t producer_partial_doubles(long long M, int C) { return (size_t)((M + 127) / 128) * 2 * (size_t)C; }

bool slice_sum_stats(const float* part, int S, float* D, long long M, int C, const FoldPlan& fp, double* partial, PartialSums* out, cudaStream_t st) {
    if (fp.vec != 4 || !aligned16(part) || !aligned16(D) || (M * C) % 4 != 0) return false;
    const int copies = fp.fused ? fp.copies_fwd : 1;
    launch(slice_sum_stats_kernel<4>, dim3(fold_grid(fp)), dim3(32, 8), 0, st, part, S, M * C, D, fp.rows, fp.cols, fold_rpc(fp), partial, C, copies);
    *out = PartialSums{partial, fp.chunks * (fp.f / copies), fp.f / copies};
    return true;
}

template <typename T>
PartialSums bn_stats(const T* y, long long M, int C, const FoldPlan& fp, double* partial, cudaStream_t st) {
    constexpr int V = VecOf<T>::N;
    if (fp.vec == V && aligned16(y)) {
        const int copies = fp.fused ? fp.copies_fwd : 1;
        launch(bn_stats_kernel<T, V>, dim3(fold_grid(fp)), dim3(32, 8), 0, st, y, fp.rows, fp.cols, fold_rpc(fp), partial, C, copies);
        return PartialSums{partial, fp.chunks * (fp.f / copies), fp.f / copies};
    }
    launch(bn_stats_kernel<T, 1>, dim3(fold_grid(fp)), dim3(32, 8), 0, st, y, fp.rows, fp.cols, fold_rpc(fp), partial, C, 1);
    return PartialSums{partial, fp.chunks * fp.f, fp.f};
}

void bn_finalize(const PartialSums& ps, long long M, int C, const float* gamma, const float* beta,
                 float eps, float momentum, float* run_mean, float* run_var, float* scale, float* shift, float* mean,
                 float* mean_lo, float* rstd, float* offset, const FinScratch& fin, cudaStream_t st) {
    if (ps.entries <= FIN_SMALL_ENTRIES)
        launch(bn_finalize_kernel<FIN_Y_SMALL>, dim3((C + FIN_X - 1) / FIN_X, 1), dim3(FIN_X, FIN_Y_SMALL), 0, st, ps.p, ps.entries / ps.fp, ps.fp, C, C * ps.fp, (double)M,
               1.0 / (double)M, M > 1 ? (double)M / (double)(M - 1) : 1.0, gamma, beta, eps, momentum, run_mean, run_var, scale, shift, mean, mean_lo, rstd, offset, fin);
    else
        launch(bn_finalize_kernel<FIN_Y>, dim3((C + FIN_X - 1) / FIN_X, fin_slices_ps(ps)), dim3(FIN_X, FIN_Y), 0, st, ps.p, ps.entries / ps.fp, ps.fp, C, C * ps.fp, (double)M,
               1.0 / (double)M, M > 1 ? (double)M / (double)(M - 1) : 1.0, gamma, beta, eps, momentum, run_mean, run_var, scale, shift, mean, mean_lo, rstd, offset, fin);
}

template <typename T>
void bn_apply(const T* y, const T* residual, T* z, long long M, int C, const FoldPlan& fp, const float* scale, const float* shift,
              const float* mean, const float* mean_lo, int act, cudaStream_t st) {
    constexpr int V = VecOf<T>::N;
    if (fp.vec == V && aligned16(y) && aligned16(residual) && aligned16(z) && aligned16(scale) && aligned16(shift) && aligned16(mean) && aligned16(mean_lo))
        launch(bn_apply_kernel<T, V>, dim3(fold_grid(fp)), dim3(32, 8), 0, st, y, residual, z, fp.rows, fp.cols, fold_rpc(fp), C, scale, shift, mean, mean_lo, act);
    else
        launch(bn_apply_kernel<T, 1>, dim3((fp.cols + 31) / 32, fp.chunks), dim3(32, 8), 0, st, y, residual, z, fp.rows, fp.cols, fold_rpc(fp), C, scale, shift, mean, mean_lo, act);
}

template <typename T>
PartialSums bn_bwd_reduce(const T* dz, const T* y, long long M, int C, const FoldPlan& fp, const float* scale, const float* shift,
                          const float* mean, const float* mean_lo, const float* rstd, int act, double* partial, cudaStream_t st) {
    constexpr int V = VecOf<T>::N;
    constexpr int W = 4;      // columns per thread: four keep the per-channel constants of a thread at a register count that leaves four blocks per SM
    if (fp.vec == V && aligned16(dz) && aligned16(y) && aligned16(scale) && aligned16(shift) && aligned16(mean) && aligned16(mean_lo) && aligned16(rstd)) {
        const int copies = fp.fused ? fp.copies_bwd : 1;
        // the plan counts column tiles of V columns per thread; with W < V (bf16) there are V / W times as many, so the rows are
        // cut into that many fewer chunks to keep the grid at the planned number of blocks (config 3: 5.050 -> 5.025 ms)
        FoldPlan q = fp;
        if (V > W) {
            const int ch = std::max(1, fp.chunks * W / V);
            const int rpc = (fp.rows + ch - 1) / ch;
            q.chunks = (fp.rows + rpc - 1) / rpc;
        }
        launch(bn_bwd_reduce_kernel<T, W>, dim3(fold_grid_w(q, W)), dim3(32, 8), 0, st, dz, y, q.rows, q.cols, fold_rpc(q), C, scale, shift, mean, mean_lo, rstd, act, partial, copies);
        return PartialSums{partial, q.chunks * (q.f / copies), q.f / copies};
    }
    // the scalar fallback keeps the plain partial layout
    launch(bn_bwd_reduce_kernel<T, 1>, dim3((fp.cols + 31) / 32, fp.chunks), dim3(32, 8), 0, st, dz, y, fp.rows, fp.cols, fold_rpc(fp), C, scale, shift, mean, mean_lo, rstd, act, partial, 1);
    return PartialSums{partial, fp.chunks * fp.f, fp.f};
}

void bn_bwd_finalize(const PartialSums& ps, long long M, int C, const float* gamma, const float* rstd,
                     float* dgamma, float* dbeta, float* coef, const FinScratch& fin, cudaStream_t st) {
    if (ps.entries <= FIN_SMALL_ENTRIES)
        launch(bn_bwd_finalize_kernel<FIN_Y_SMALL>, dim3((C + FIN_X - 1) / FIN_X, 1), dim3(FIN_X, FIN_Y_SMALL), 0, st, ps.p, ps.entries / ps.fp, ps.fp, C, C * ps.fp,
           1.0 / (double)M, gamma, rstd, dgamma, dbeta, coef, fin);
    else
        launch(bn_bwd_finalize_kernel<FIN_Y>, dim3((C + FIN_X - 1) / FIN_X, fin_slices_ps(ps)), dim3(FIN_X, FIN_Y), 0, st, ps.p, ps.entries / ps.fp, ps.fp, C, C * ps.fp,
           1.0 / (double)M, gamma, rstd, dgamma, dbeta, coef, fin);
}

template <typename T>
void bn_bwd_apply(const T* dz, const T* y, const T* addend, T* dy, long long M, int C, const FoldPlan& fp, const float* scale, const float* shift,
                  const float* mean, const float* mean_lo, const float* rstd, const float* coef, int act, cudaStream_t st) {
    constexpr int V = VecOf<T>::N;
    constexpr int W = 4;      // columns per thread: four keep the per-channel constants of a thread at a register count that leaves four blocks per SM
    if (fp.vec == V && aligned16(dz) && aligned16(y) && aligned16(addend) && aligned16(dy) && aligned16(scale) && aligned16(shift) && aligned16(mean) &&
        aligned16(mean_lo) && aligned16(rstd) && aligned16(coef))
        launch(bn_bwd_apply_kernel<T, W>, dim3(fold_grid_w(fp, W)), dim3(32, 8), 0, st, dz, y, addend, dy, fp.rows, fp.cols, fold_rpc(fp), C, scale, shift, mean, mean_lo, rstd, coef, act);
    else
        launch(bn_bwd_apply_kernel<T, 1>, dim3((fp.cols + 31) / 32, fp.chunks), dim3(32, 8), 0, st, dz, y, addend, dy, fp.rows, fp.cols, fold_rpc(fp), C, scale, shift, mean, mean_lo, rstd, coef, act);
}

template <typename T>
void act_bias_bwd(const T* dout, const T* out, T* dpre, long long M, int C, int act, const FoldPlan& fp, double* partial,
                  float* dbias, const FinScratch& fin, cudaStream_t st) {
    constexpr int V = VecOf<T>::N;
    if (fp.vec == V && aligned16(dout) && aligned16(out) && aligned16(dpre))
        launch(act_bias_bwd_kernel<T, V>, dim3(fold_grid(fp)), dim3(32, 8), 0, st, dout, out, dpre, fp.rows, fp.cols, fold_rpc(fp), act, partial);
    else
        launch(act_bias_bwd_kernel<T, 1>, dim3((fp.cols + 31) / 32, fp.chunks), dim3(32, 8), 0, st, dout, out, dpre, fp.rows, fp.cols, fold_rpc(fp), act, partial);
    if (dbias) launch(colsum_finalize_kernel, dim3((C + FIN_X - 1) / FIN_X, fin_slices(fp)), dim3(FIN_X, FIN_Y), 0, st, partial, fp.chunks, fp.f, C, fp.cols, dbias, fin);
}

template <typename T>
void act_fwd(const T* x, T* y, long long n, int act, cudaStream_t st) {
    constexpr int V = VecOf<T>::N;
    if (n % V == 0 && aligned16(x) && aligned16(y)) launch(act_fwd_kernel<T, V>, dim3(flat_blocks(n / V, 256)), dim3(256), 0, st, x, y, n / V, act);
    else launch(act_fwd_kernel<T, 1>, dim3(flat_blocks(n, 256)), dim3(256), 0, st, x, y, n, act);
}

template <typename T>
void act_bwd(const T* dout, const T* x, const T* addend, T* dx, long long n, int act, cudaStream_t st) {
    constexpr int V = VecOf<T>::N;
    if (n % V == 0 && aligned16(dout) && aligned16(x) && aligned16(addend) && aligned16(dx))
        launch(act_bwd_kernel<T, V>, dim3(flat_blocks(n / V, 256)), dim3(256), 0, st, dout, x, addend, dx, n / V, act);
    else launch(act_bwd_kernel<T, 1>, dim3(flat_blocks(n, 256)), dim3(256), 0, st, dout, x, addend, dx, n, act);
}

// log2 of the tile width: the largest power of two <= min(8, width)
static inline int dw_tile_shift(int width) { return width >= 8 ? 3 : width >= 4 ? 2 : width >= 2 ? 1 : 0; }

// Row chunks per image for the row-marching kernels.  A block walks groups of 32 slots (blockIdx.x, + gridDim.x, ...);
// `resident_blocks` blocks are resident at once.  Longer walks re-load fewer halo rows, shorter ones balance the blocks better.
struct Dw3Plan { int RH, HC; unsigned gx, gy; long long groups; };
static Dw3Plan plan_dw3(const ConvGeom& g, int resident_blocks) {
    const int strips_w = (g.W + 3) / 4, cgroups = (g.Cin / 4 + 7) / 8;
    const long long slots_x = std::max(1, resident_blocks / cgroups);
    auto groups = [&](int hc) { return ((long long)g.N * hc * strips_w + 31) / 32; };
    // chunks of at most eight rows (a quarter more rows loaded than computed, and groups enough that the blocks' shares
    // differ little); shorter ones, down to two rows, while the blocks would not fill the machine (small maps: latency counts)
    int best = 1;
    while ((g.H + best - 1) / best > 8) best *= 2;
    while (groups(best) * cgroups < resident_blocks && (g.H + 2 * best - 1) / (2 * best) >= 2) best *= 2;
    Dw3Plan p;
    p.RH = (g.H + best - 1) / best;
    p.HC = (g.H + p.RH - 1) / p.RH;
    p.groups = groups(p.HC);
    p.gx = (unsigned)std::min<long long>(p.groups, slots_x);
    p.gy = (unsigned)cgroups;
    return p;
}
// The same for the stride-2 kernels: strips of two output columns, chunks of output rows.
static Dw3Plan plan_dw3s2(const ConvGeom& g, int resident_blocks) {
    const int strips_w = (g.Wo + 1) / 2, cgroups = (g.Cin / 4 + 7) / 8;
    const long long slots_x = std::max(1, resident_blocks / cgroups);
    auto groups = [&](int hc) { return ((long long)g.N * hc * strips_w + 31) / 32; };
    int best = 1;
    while ((g.Ho + best - 1) / best > 8) best *= 2;
    while (groups(best) * cgroups < resident_blocks && (g.Ho + 2 * best - 1) / (2 * best) >= 2) best *= 2;
    Dw3Plan p;
    p.RH = (g.Ho + best - 1) / best;
    p.HC = (g.Ho + p.RH - 1) / p.RH;
    p.groups = groups(p.HC);
    // a block leaves one entry of partial sums: no more blocks than the statistics buffers of a [M][C] tensor hold
    const long long room = ((long long)g.N * g.Ho * g.Wo + 127) / 128;
    p.gx = (unsigned)std::max<long long>(1, std::min(std::min<long long>(p.groups, slots_x), room));
    p.gy = (unsigned)cgroups;
    return p;
}
static bool dw_s2_shape(const ConvGeom& g) { return g.stride == 2 && g.ph == 1 && g.pw == 1 && g.kh == 3 && g.kw == 3 && g.Cin % 4 == 0; }
// FTP_DW_ROWS2: the stride-2 row kernels: 0 never, 1 float tensors only, 2 always (default)
static bool dw_rows2_enabled(size_t elem_bytes) {
    static int on = -1;
    if (on < 0) { const char* e = std::getenv("FTP_DW_ROWS2"); on = e ? std::atoi(e) : 2; }
    return on == 2 || (on == 1 && elem_bytes == 4);
}
// FTP_DW_ROWS: 0 never, 1 float tensors only (default: on bf16 tensors the two separate kernels, one of them on the
// second stream, are faster), 2 always
static bool dw_rows_enabled(size_t elem_bytes) {
    static int on = -1;
    if (on < 0) { const char* e = std::getenv("FTP_DW_ROWS"); on = e ? std::atoi(e) : 1; }
    return on == 2 || (on == 1 && elem_bytes == 4);
}

template <typename T>
void dwconv_fwd(const T* x, const float* w, T* y, const ConvGeom& g, cudaStream_t st, const ColStatsReq* stats, const BnXform* x_xform) {
    constexpr int V = VecOf<T>::N;
    const int tws = dw_tile_shift(g.Wo);
    const unsigned tiles = (unsigned)(((g.Wo + (1 << tws) - 1) >> tws) * (((long long)g.N * g.Ho + (64 >> tws) - 1) / (64 >> tws)));
    if (stats) stats->out->entries = 0;
    const bool xf = x_xform != nullptr;
    const BnXform xv = xf ? *x_xform : BnXform{nullptr, nullptr, nullptr, 0.f, 0.f};
    const bool xf_vec = !xf || (aligned16(xv.mean) && aligned16(xv.scale) && aligned16(xv.offset));
    if (dw_rows_enabled(sizeof(T)) && g.stride == 1 && g.ph == 1 && g.pw == 1 && can_vec<T>(g.Cin, x, y) && aligned16(w) && xf_vec) {
        const Dw3Plan pl = plan_dw3(g, (xf ? 1 : 2) * sm_count());         // resident blocks per SM: see the kernel's launch bounds
        const dim3 grid(pl.gx, pl.gy);
        double* sp = stats ? stats->partial : nullptr;
        if (stats) {
            if (xf) launch(dw3_fwd_rows_kernel<T, true, true>, grid, dim3(256), 0, st, x, w, y, g.N, g.H, g.W, g.Cin, pl.RH, pl.HC, sp, xv);
            else launch(dw3_fwd_rows_kernel<T, false, true>, grid, dim3(256), 0, st, x, w, y, g.N, g.H, g.W, g.Cin, pl.RH, pl.HC, sp, xv);
            *stats->out = PartialSums{stats->partial, (int)grid.x, 1};
        } else if (xf) launch(dw3_fwd_rows_kernel<T, true, false>, grid, dim3(256), 0, st, x, w, y, g.N, g.H, g.W, g.Cin, pl.RH, pl.HC, sp, xv);
        else launch(dw3_fwd_rows_kernel<T, false, false>, grid, dim3(256), 0, st, x, w, y, g.N, g.H, g.W, g.Cin, pl.RH, pl.HC, sp, xv);
        return;
    }
    if (dw_rows2_enabled(sizeof(T)) && dw_s2_shape(g) && can_vec<T>(g.Cin, x, y) && aligned16(w) && xf_vec) {
        const Dw3Plan pl = plan_dw3s2(g, 2 * sm_count());
        const dim3 grid(pl.gx, pl.gy);
        double* sp = stats ? stats->partial : nullptr;
        if (stats) {
            if (xf) launch(dw3s2_fwd_rows_kernel<T, true, true>, grid, dim3(256), 0, st, x, w, y, g.N, g.H, g.W, g.Cin, g.Ho, g.Wo, pl.RH, pl.HC, sp, xv);
            else launch(dw3s2_fwd_rows_kernel<T, false, true>, grid, dim3(256), 0, st, x, w, y, g.N, g.H, g.W, g.Cin, g.Ho, g.Wo, pl.RH, pl.HC, sp, xv);
            *stats->out = PartialSums{stats->partial, (int)grid.x, 1};
        } else if (xf) launch(dw3s2_fwd_rows_kernel<T, true, false>, grid, dim3(256), 0, st, x, w, y, g.N, g.H, g.W, g.Cin, g.Ho, g.Wo, pl.RH, pl.HC, sp, xv);
        else launch(dw3s2_fwd_rows_kernel<T, false, false>, grid, dim3(256), 0, st, x, w, y, g.N, g.H, g.W, g.Cin, g.Ho, g.Wo, pl.RH, pl.HC, sp, xv);
        return;
    }
    if (g.stride == 1 && g.ph == 1 && g.pw == 1 && can_vec<T>(g.Cin, x, y) && aligned16(w) && xf_vec) {
        const long long strips = (long long)g.N * g.H * ((g.W + 3) / 4);
        const dim3 grid((unsigned)((strips + 31) / 32), (g.Cin / 4 + 7) / 8);
        // four channels per thread for either type: eight lanes of a block then cover 32 channels, which every layer has
        if (stats) {
            if (xf) launch(dw_strip_kernel<T, 4, 0, 1, true>, grid, dim3(256), 0, st, x, w, (const T*)nullptr, y, g.N, g.H, g.W, g.Cin, stats->partial, xv);
            else launch(dw_strip_kernel<T, 4, 0, 1, false>, grid, dim3(256), 0, st, x, w, (const T*)nullptr, y, g.N, g.H, g.W, g.Cin, stats->partial, xv);
            *stats->out = PartialSums{stats->partial, (int)grid.x, 1};
        } else if (xf) launch(dw_strip_kernel<T, 4, 0, 0, true>, grid, dim3(256), 0, st, x, w, (const T*)nullptr, y, g.N, g.H, g.W, g.Cin, (double*)nullptr, xv);
        else launch(dw_strip_kernel<T, 4, 0, 0, false>, grid, dim3(256), 0, st, x, w, (const T*)nullptr, y, g.N, g.H, g.W, g.Cin, (double*)nullptr, xv);
        return;
    }
    if (can_vec<T>(g.Cin, x, y) && aligned16(w) && xf_vec) {
        const dim3 grid(tiles, (g.Cin / V + 7) / 8);
        if (xf) launch(dw_fwd_kernel<T, V, true>, grid, dim3(256), 0, st, x, w, y, g, tws, xv);
        else launch(dw_fwd_kernel<T, V, false>, grid, dim3(256), 0, st, x, w, y, g, tws, xv);
    } else {
        const dim3 grid(tiles, (g.Cin + 7) / 8);
        if (xf) launch(dw_fwd_kernel<T, 1, true>, grid, dim3(256), 0, st, x, w, y, g, tws, xv);
        else launch(dw_fwd_kernel<T, 1, false>, grid, dim3(256), 0, st, x, w, y, g, tws, xv);
    }
}

template <typename T>
void dwconv_dgrad(const T* dy, const float* w, const T* addend, T* dx, const ConvGeom& g, cudaStream_t st) {
    constexpr int V = VecOf<T>::N;
    const int tws = dw_tile_shift(g.W);
    const unsigned tiles = (unsigned)(((g.W + (1 << tws) - 1) >> tws) * (((long long)g.N * g.H + (64 >> tws) - 1) / (64 >> tws)));
    if (g.stride == 1 && g.ph == 1 && g.pw == 1 && can_vec<T>(g.Cin, dy, addend, dx) && aligned16(w)) {
        const long long strips = (long long)g.N * g.H * ((g.W + 3) / 4);
        launch(dw_strip_kernel<T, 4, 1, 0, false>, dim3((unsigned)((strips + 31) / 32), (g.Cin / 4 + 7) / 8), dim3(256), 0, st, dy, w, addend, dx, g.N, g.H, g.W, g.Cin, (double*)nullptr,
               BnXform{nullptr, nullptr, nullptr, 0.f, 0.f});
        return;
    }
    if (can_vec<T>(g.Cin, dy, addend, dx) && aligned16(w)) {
        const dim3 grid(tiles, (g.Cin / V + 7) / 8);
        if (g.stride == 2) launch(dw_dgrad_kernel<T, V, 2>, grid, dim3(256), 0, st, dy, w, addend, dx, g, tws);
        else if (g.stride == 1) launch(dw_dgrad_kernel<T, V, 1>, grid, dim3(256), 0, st, dy, w, addend, dx, g, tws);
        else launch(dw_dgrad_kernel<T, V, 0>, grid, dim3(256), 0, st, dy, w, addend, dx, g, tws);
    } else launch(dw_dgrad_kernel<T, 1, 0>, dim3(tiles, (g.Cin + 7) / 8), dim3(256), 0, st, dy, w, addend, dx, g, tws);
}

static FoldPlan plan_dw_wgrad(const ConvGeom& g, int elem_bytes) {
    return make_fold((long long)g.N * g.Ho * g.Wo, g.Cin, elem_bytes);
}

// strip kernel: number of blocks along the strips (each block walks strips with that stride)
static inline int dw_wgrad_strip_blocks(const ConvGeom& g, int V, bool rows_variant) {
    const long long strips = (long long)g.N * g.H * ((g.W + 3) / 4);
    const int cgroups = (g.Cin / V + 7) / 8;
    const int per_block = rows_variant ? DW_WG_STRIPS : 32;
    long long gx = ((rows_variant ? 8LL : 6LL) * sm_count() + cgroups - 1) / cgroups;
    const long long most = (strips + per_block - 1) / per_block;
    if (gx > most) gx = most;
    return (int)(gx < 1 ? 1 : gx);
}

size_t dwconv_wgrad_scratch_floats(const ConvGeom& g) {
    const FoldPlan a = plan_dw_wgrad(g, 4), b = plan_dw_wgrad(g, 2);
    size_t n = std::max((size_t)a.chunks * 9 * a.cols, (size_t)b.chunks * 9 * b.cols);
    if (g.Cin % 4 == 0 && g.stride == 1) n = std::max(n, (size_t)plan_dw3(g, sm_count()).gx * 9 * g.Cin);
    if (dw_s2_shape(g)) n = std::max(n, (size_t)plan_dw3s2(g, sm_count()).gx * 9 * g.Cin);
    if (g.Cin % 4 == 0) n = std::max(n, (size_t)std::max(dw_wgrad_strip_blocks(g, 4, false), dw_wgrad_strip_blocks(g, 4, true)) * 9 * g.Cin);
    return n;
}

template <typename T>
void dwconv_wgrad(const T* x, const T* dy, float* dw, float* scratch, const ConvGeom& g, const FinScratch& fin, cudaStream_t st, const BnXform* x_xform) {
    constexpr int V = VecOf<T>::N;
    const bool xf = x_xform != nullptr;
    const BnXform xv = xf ? *x_xform : BnXform{nullptr, nullptr, nullptr, 0.f, 0.f};
    const bool xf_vec = !xf || (aligned16(xv.mean) && aligned16(xv.scale) && aligned16(xv.offset));
    // four channels per thread for either type: with eight bf16 channels the nine accumulators would leave too few warps per SM
    if (g.stride == 1 && g.ph == 1 && g.pw == 1 && can_vec<T>(g.Cin, x, dy) && xf_vec) {
        constexpr int SV = 4;
        constexpr bool rows_variant = sizeof(T) == 2;
        const int gx = dw_wgrad_strip_blocks(g, SV, rows_variant);
        const dim3 grid(gx, (g.Cin / SV + 7) / 8);
        if (rows_variant) {
            if (xf) launch(dw_wgrad_rows_kernel<T, SV, true>, grid, dim3(256), 0, st, x, dy, scratch, g.N, g.H, g.W, g.Cin, xv);
            else launch(dw_wgrad_rows_kernel<T, SV, false>, grid, dim3(256), 0, st, x, dy, scratch, g.N, g.H, g.W, g.Cin, xv);
        } else {
            if (xf) launch(dw_wgrad_strip_kernel<T, SV, true>, grid, dim3(256), 0, st, x, dy, scratch, g.N, g.H, g.W, g.Cin, xv);
            else launch(dw_wgrad_strip_kernel<T, SV, false>, grid, dim3(256), 0, st, x, dy, scratch, g.N, g.H, g.W, g.Cin, xv);
        }
        if (gx <= DW_FIN_SMALL) {
            launch(dw_wgrad_finalize_small_kernel, dim3((g.Cin + 31) / 32, 9), dim3(32, 8), 0, st, (const float*)scratch, gx, 1, g.Cin, g.Cin, dw);
            return;
        }
        int slices = gx / (4 * FIN_Y);
        slices = slices < 1 ? 1 : (slices > FIN_GMAX ? FIN_GMAX : slices);
        launch(dw_wgrad_finalize_kernel, dim3((g.Cin + FIN_X - 1) / FIN_X, slices, 9), dim3(FIN_X, FIN_Y), 0, st, (const float*)scratch, gx, 1, g.Cin, g.Cin, dw, fin);
        return;
    }
    FoldPlan fp = plan_dw_wgrad(g, (int)sizeof(T));
    const int rpc = fold_rpc(fp);
    if (fp.vec == V && aligned16(x) && aligned16(dy) && xf_vec) {
        if (xf) launch(dw_wgrad_kernel<T, V, true>, dim3(fold_grid(fp)), dim3(32, 8), 0, st, x, dy, scratch, g, fp.rows, fp.cols, fp.f, rpc, xv);
        else launch(dw_wgrad_kernel<T, V, false>, dim3(fold_grid(fp)), dim3(32, 8), 0, st, x, dy, scratch, g, fp.rows, fp.cols, fp.f, rpc, xv);
    } else {
        const dim3 grid((fp.cols + 31) / 32, fp.chunks);
        if (xf) launch(dw_wgrad_kernel<T, 1, true>, grid, dim3(32, 8), 0, st, x, dy, scratch, g, fp.rows, fp.cols, fp.f, rpc, xv);
        else launch(dw_wgrad_kernel<T, 1, false>, grid, dim3(32, 8), 0, st, x, dy, scratch, g, fp.rows, fp.cols, fp.f, rpc, xv);
    }
    if (fp.chunks * fp.f <= DW_FIN_SMALL) launch(dw_wgrad_finalize_small_kernel, dim3((g.Cin + 31) / 32, 9), dim3(32, 8), 0, st, (const float*)scratch, fp.chunks, fp.f, g.Cin, fp.cols, dw);
    else launch(dw_wgrad_finalize_kernel, dim3((g.Cin + FIN_X - 1) / FIN_X, fin_slices(fp), 9), dim3(FIN_X, FIN_Y), 0, st, scratch, fp.chunks, fp.f, g.Cin, fp.cols, dw, fin);
}

size_t dwconv_bwd_stats_doubles(const ConvGeom& g) {
    if (dw_s2_shape(g)) return (size_t)plan_dw3s2(g, sm_count()).gx * 2 * g.Cin;
    return g.Cin % 4 == 0 && g.stride == 1 ? (size_t)plan_dw3(g, sm_count()).gx * 2 * g.Cin : 0;
}

template <typename T>
bool dwconv_bwd_fused(const T* x, const T* dy, const float* w, const T* addend, T* dx, float* dw, float* scratch, const ConvGeom& g, const FinScratch& fin,
                      cudaStream_t st, const BnXform* x_xform, const BnBwdSumsReq* sums, cudaStream_t fin_st, cudaEvent_t fin_fork) {
    const bool xf = x_xform != nullptr;
    const BnXform xv = xf ? *x_xform : BnXform{nullptr, nullptr, nullptr, 0.f, 0.f};
    const bool xf_vec = !xf || (aligned16(xv.mean) && aligned16(xv.scale) && aligned16(xv.offset));
    if (sums) sums->out->entries = 0;
    const bool bst = xf && sums && dx && aligned16(sums->rstd);
    const bool s2 = dw_rows2_enabled(sizeof(T)) && dw_s2_shape(g);
    if (s2 && !(can_vec<T>(g.Cin, x, dy, addend, dx) && aligned16(w) && xf_vec)) return false;
    if (!s2 && !(dw_rows_enabled(sizeof(T)) && g.stride == 1 && g.ph == 1 && g.pw == 1 && can_vec<T>(g.Cin, x, dy, addend, dx) && g.Cin % 4 == 0 && xf_vec)) return false;
    const Dw3Plan pl = s2 ? plan_dw3s2(g, sm_count()) : plan_dw3(g, sm_count());
    const dim3 grid(pl.gx, pl.gy);
    if (s2) {
        if (bst) {
            launch(dw3s2_bwd_rows_kernel<T, true, true>, grid, dim3(256), 0, st, x, dy, w, addend, dx, scratch, g.N, g.H, g.W, g.Cin, g.Ho, g.Wo, pl.RH, pl.HC, xv, sums->rstd, sums->partial);
            *sums->out = PartialSums{sums->partial, (int)grid.x, 1};
        } else if (xf) launch(dw3s2_bwd_rows_kernel<T, true, false>, grid, dim3(256), 0, st, x, dy, w, addend, dx, scratch, g.N, g.H, g.W, g.Cin, g.Ho, g.Wo, pl.RH, pl.HC, xv, (const float*)nullptr, (double*)nullptr);
        else launch(dw3s2_bwd_rows_kernel<T, false, false>, grid, dim3(256), 0, st, x, dy, w, addend, dx, scratch, g.N, g.H, g.W, g.Cin, g.Ho, g.Wo, pl.RH, pl.HC, xv, (const float*)nullptr, (double*)nullptr);
    } else if (bst) {
        launch(dw3_bwd_rows_kernel<T, true, true>, grid, dim3(256), 0, st, x, dy, w, addend, dx, scratch, g.N, g.H, g.W, g.Cin, pl.RH, pl.HC, xv, sums->rstd, sums->partial);
        *sums->out = PartialSums{sums->partial, (int)grid.x, 1};
    } else if (xf) launch(dw3_bwd_rows_kernel<T, true, false>, grid, dim3(256), 0, st, x, dy, w, addend, dx, scratch, g.N, g.H, g.W, g.Cin, pl.RH, pl.HC, xv, (const float*)nullptr, (double*)nullptr);
    else launch(dw3_bwd_rows_kernel<T, false, false>, grid, dim3(256), 0, st, x, dy, w, addend, dx, scratch, g.N, g.H, g.W, g.Cin, pl.RH, pl.HC, xv, (const float*)nullptr, (double*)nullptr);
    const int gx = (int)pl.gx;
    // the sums over the blocks' weight-gradient partials feed only the update: the caller may give them another stream
    if (fin_st == nullptr) fin_st = st;
    if (fin_st != st) { cudaEventRecord(fin_fork, st); cudaStreamWaitEvent(fin_st, fin_fork, 0); }
    if (gx <= DW_FIN_SMALL) launch(dw_wgrad_finalize_small_kernel, dim3((g.Cin + 31) / 32, 9), dim3(32, 8), 0, fin_st, (const float*)scratch, gx, 1, g.Cin, g.Cin, dw);
    else {
        int slices = gx / (4 * FIN_Y);
        slices = slices < 1 ? 1 : (slices > FIN_GMAX ? FIN_GMAX : slices);
        launch(dw_wgrad_finalize_kernel, dim3((g.Cin + FIN_X - 1) / FIN_X, slices, 9), dim3(FIN_X, FIN_Y), 0, fin_st, (const float*)scratch, gx, 1, g.Cin, g.Cin, dw, fin);
    }
    return true;
}

template <typename T>
void maxpool_fwd(const T* x, T* y, int N, int H, int W, int C, cudaStream_t st) {
    constexpr int V = VecOf<T>::N;
    const long long pix = (long long)N * (H / 2) * (W / 2);
    if (can_vec<T>(C, x, y)) launch(maxpool_fwd_kernel<T, V>, dim3(flat_blocks(pix * (C / V), 256)), dim3(256), 0, st, x, y, H, W, C, pix * (C / V));
    else launch(maxpool_fwd_kernel<T, 1>, dim3(flat_blocks(pix * C, 256)), dim3(256), 0, st, x, y, H, W, C, pix * C);
}

template <typename T>
void maxpool_bwd(const T* dy, const T* x, T* dx, int N, int H, int W, int C, cudaStream_t st) {
    constexpr int V = VecOf<T>::N;
    const long long pix = (long long)N * (H / 2) * (W / 2);
    if ((H & 1) || (W & 1)) cudaMemsetAsync(dx, 0, (size_t)N * H * W * C * sizeof(T), st);   // odd edge gets no gradient
    if (can_vec<T>(C, dy, x, dx)) launch(maxpool_bwd_kernel<T, V>, dim3(flat_blocks(pix * (C / V), 256)), dim3(256), 0, st, dy, x, dx, H, W, C, pix * (C / V));
    else launch(maxpool_bwd_kernel<T, 1>, dim3(flat_blocks(pix * C, 256)), dim3(256), 0, st, dy, x, dx, H, W, C, pix * C);
}

template <typename T>
void gap_fwd(const T* x, T* y, int N, int HW, int C, cudaStream_t st) {
    constexpr int V = VecOf<T>::N;
    if (can_vec<T>(C, x, y)) { const long long t = (long long)N * (C / V); launch(gap_fwd_kernel<T, V>, dim3((unsigned)((t + 255) / 256)), dim3(256), 0, st, x, y, HW, C, t); }
    else { const long long t = (long long)N * C; launch(gap_fwd_kernel<T, 1>, dim3((unsigned)((t + 255) / 256)), dim3(256), 0, st, x, y, HW, C, t); }
}

template <typename T>
void gap_bwd(const T* dy, T* dx, int N, int HW, int C, cudaStream_t st) {
    constexpr int V = VecOf<T>::N;
    if (can_vec<T>(C, dy, dx)) { const long long t = (long long)N * HW * (C / V); launch(gap_bwd_kernel<T, V>, dim3(flat_blocks(t, 256)), dim3(256), 0, st, dy, dx, HW, C, t); }
    else { const long long t = (long long)N * HW * C; launch(gap_bwd_kernel<T, 1>, dim3(flat_blocks(t, 256)), dim3(256), 0, st, dy, dx, HW, C, t); }
}

void softmax_ce(const float* logits, const int32_t* labels, int N, int classes, float* per_sample, float* dlogits,
                float* loss, cudaStream_t st) {
    launch(softmax_ce_kernel, dim3(N), dim3(128), 0, st, logits, labels, N, classes, per_sample, dlogits);
    launch(loss_mean_kernel, dim3(1), dim3(32), 0, st, per_sample, N, loss);
}

void sgd_update(float* w, const float* g, float* m, long long n, float lr, float mu, float wd, int first,
                __nv_bfloat16* shadow, float* lo, float* snap_dev, float* snap_host, cudaStream_t st) {
    const bool v = n >= 4 && aligned16(w) && aligned16(g) && aligned16(m) && aligned16(lo) && aligned16(snap_dev) && aligned16(snap_host);
    if (v) launch(sgd_kernel<4>, dim3(flat_blocks(n / 4, 256)), dim3(256), 0, st, w, g, m, n / 4, (int)(n % 4), lr, mu, wd, first, shadow, lo, snap_dev, snap_host);
    else launch(sgd_kernel<1>, dim3(flat_blocks(n, 256)), dim3(256), 0, st, w, g, m, n, 0, lr, mu, wd, first, shadow, lo, snap_dev, snap_host);
}

void mean_f32(const MeanSources& src, float* dst, long long count, cudaStream_t st) {
    if (count > 0) launch(mean_f32_kernel, dim3(flat_blocks(count, 256)), dim3(256), 0, st, src, dst, count);
}

void tf32_lo(const float* w, float* lo, long long n, cudaStream_t st) {
    launch(tf32_lo_kernel, dim3(flat_blocks(n, 256)), dim3(256), 0, st, w, lo, n);
}

void transpose_split_f32(const TransposeEntryDev* table, int n, int tile_base, int tiles, const float* w, float* wt, float* wtl, cudaStream_t st) {
    if (tiles > 0) launch(transpose_split_f32_kernel, dim3(tiles), dim3(32, 8), 0, st, table, n, tile_base, w, wt, wtl);
}

void transpose_bf16_batched(const TransposeEntryDev* table, int n, int tile_base, int tiles, const float* w, __nv_bfloat16* wt, cudaStream_t st) {
    if (tiles > 0) launch(transpose_bf16_batched_kernel, dim3(tiles), dim3(32, 8), 0, st, table, n, tile_base, w, wt);
}

void bf16_to_f32(const __nv_bfloat16* src, float* dst, long long n, cudaStream_t st) {
    launch(bf16_to_f32_kernel, dim3(flat_blocks(n, 256)), dim3(256), 0, st, src, dst, n);
}

void f32_to_bf16(const float* src, __nv_bfloat16* dst, long long n, cudaStream_t st) {
    launch(f32_to_bf16_kernel, dim3(flat_blocks(n, 256)), dim3(256), 0, st, src, dst, n);
}

#define FTP_INSTANTIATE(T)                                                                                              \
    template PartialSums bn_stats<T>(const T*, long long, int, const FoldPlan&, double*, cudaStream_t);                          \
    template void bn_apply<T>(const T*, const T*, T*, long long, int, const FoldPlan&, const float*, const float*, const float*, \
                              const float*, int, cudaStream_t);                                                            \
    template PartialSums bn_bwd_reduce<T>(const T*, const T*, long long, int, const FoldPlan&, const float*, const float*,         \
                                   const float*, const float*, const float*, int, double*, cudaStream_t);                  \
    template void bn_bwd_apply<T>(const T*, const T*, const T*, T*, long long, int, const FoldPlan&, const float*, const float*, \
                                  const float*, const float*, const float*, const float*, int, cudaStream_t);              \
    template void act_bias_bwd<T>(const T*, const T*, T*, long long, int, int, const FoldPlan&, double*, float*,            \
                                  const FinScratch&, cudaStream_t);                                                                           \
    template void act_fwd<T>(const T*, T*, long long, int, cudaStream_t);                                                   \
    template void act_bwd<T>(const T*, const T*, const T*, T*, long long, int, cudaStream_t);                               \
    template void dwconv_fwd<T>(const T*, const float*, T*, const ConvGeom&, cudaStream_t, const ColStatsReq*, const BnXform*); \
    template void dwconv_dgrad<T>(const T*, const float*, const T*, T*, const ConvGeom&, cudaStream_t);                     \
    template void dwconv_wgrad<T>(const T*, const T*, float*, float*, const ConvGeom&, const FinScratch&, cudaStream_t, const BnXform*); \
    template bool dwconv_bwd_fused<T>(const T*, const T*, const float*, const T*, T*, float*, float*, const ConvGeom&, const FinScratch&, cudaStream_t, const BnXform*, const BnBwdSumsReq*, cudaStream_t, cudaEvent_t); \
    template void maxpool_fwd<T>(const T*, T*, int, int, int, int, cudaStream_t);                                           \
    template void maxpool_bwd<T>(const T*, const T*, T*, int, int, int, int, cudaStream_t);                                 \
    template void gap_fwd<T>(const T*, T*, int, int, int, cudaStream_t);                                                    \
    template void gap_bwd<T>(const T*, T*, int, int, int, cudaStream_t);

FTP_INSTANTIATE(float)
FTP_INSTANTIATE(__nv_bfloat16)

}  // namespace ftp
