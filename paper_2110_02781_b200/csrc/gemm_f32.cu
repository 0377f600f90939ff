// SIMT contractions: dense convolution (incl. 1x1 / FC / conv1d) forward, data gradient and
// weight gradient as implicit GEMMs with float accumulation.  They serve the shapes the tensor-core
// kernels (split-tf32 for float tensors, bf16) do not take: spatial kernels of float models, 3 input
// channels, ragged channel counts, bias or activation fused into the convolution, the classifier.
// Instantiated for float and for bfloat16 tensors.
//
// Tiling: 256 threads compute a 128 x BN tile of the output with an 8 x (BN/16) register
// micro-tile per thread; the reduction dimension is walked 16 at a time through two
// shared-memory buffers, the next tile's global loads being issued before the current tile's
// math.  The activation operand is gathered (im2col on the fly) with 16-byte loads whenever the
// channel count allows; rows are output pixels (forward), input pixels (data gradient) or
// reduction steps (weight gradient).
#include "kernels.h"
#include "launch.cuh"

namespace ftp {
namespace {

constexpr int BK = 16, NT = 256;

// four / one consecutive elements as floats
__device__ __forceinline__ float4 ldg4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ float4 ldg4(const __nv_bfloat16* p) {
    const uint2 u = __ldg(reinterpret_cast<const uint2*>(p));
    return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16), __uint_as_float(u.y & 0xffff0000u));
}
__device__ __forceinline__ float ldg1(const float* p) { return __ldg(p); }
__device__ __forceinline__ float ldg1(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void st4(float* p, float a, float b, float c, float d) { *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d); }
__device__ __forceinline__ void st4(__nv_bfloat16* p, float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<const unsigned*>(&lo), *reinterpret_cast<const unsigned*>(&hi));
}
__device__ __forceinline__ void st2(float* p, float a, float b) { *reinterpret_cast<float2*>(p) = make_float2(a, b); }
__device__ __forceinline__ void st2(__nv_bfloat16* p, float a, float b) { *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(a, b); }
__device__ __forceinline__ void st1(float* p, float a) { *p = a; }
__device__ __forceinline__ void st1(__nv_bfloat16* p, float a) { *p = __float2bfloat16_rn(a); }

template <typename T>
struct GemmP {
    const T* A;            // gathered operand: x (forward) or dy (data gradient)
    const T* B;            // weights [kh*kw][Cin][Cout]
    const float* bias;     // forward only, nullable
    const T* addend;       // nullable, shaped like D
    T* D;
    int M, Kg, Cd;         // GEMM rows, reduction length, output columns
    int Hs, Ws, Cs;        // source tensor: spatial dims and channels
    int Hd, Wd;            // destination tensor spatial dims
    int kh, kw, stride, ph, pw;
    int act, vecA, vecB, alignD, pointwise;
    int kt_per;            // reduction tiles per z-slice (split over K: slice z writes its partial at D + z*M*Cd)
};

struct RowInfo {
    int nb, hb, wb;        // n * Hs * Ws, and the row's base coordinates in the source
    bool ok;
};

template <int MODE, typename T>
__device__ __forceinline__ RowInfo make_row(const GemmP<T>& p, int m) {
    RowInfo r;
    r.ok = m < p.M;
    const int hw = p.Hd * p.Wd;
    const int n = m / hw, rem = m - n * hw;
    const int hd = rem / p.Wd, wd = rem - hd * p.Wd;
    r.nb = n * p.Hs * p.Ws;
    if (MODE == 0) { r.hb = hd * p.stride - p.ph; r.wb = wd * p.stride - p.pw; }
    else { r.hb = hd + p.ph; r.wb = wd + p.pw; }
    return r;
}

// Offset (in floats) of source element for row `ri` and tap (r, s), channel c; -1 if it is padding.
template <int MODE, typename T>
__device__ __forceinline__ long long src_offset(const GemmP<T>& p, const RowInfo& ri, int r, int s, int c) {
    int hs, ws;
    if (MODE == 0) {
        hs = ri.hb + r; ws = ri.wb + s;
        if (hs < 0 || hs >= p.Hs || ws < 0 || ws >= p.Ws) return -1;
    } else {
        const int th = ri.hb - r, tw = ri.wb - s;
        if (th < 0 || tw < 0) return -1;
        hs = th / p.stride; ws = tw / p.stride;
        if (hs * p.stride != th || ws * p.stride != tw || hs >= p.Hs || ws >= p.Ws) return -1;
    }
    return ((long long)(ri.nb + hs * p.Ws + ws)) * p.Cs + c;
}

__device__ __forceinline__ float apply_act(float v, int act) {
    if (act == 1) return fmaxf(v, 0.f);
    if (act == 2) return fminf(fmaxf(v, 0.f), 6.f);
    return v;
}

template <int BM, int BN, int MODE, typename T>
__global__ void __launch_bounds__(NT) conv_gemm_kernel(const GemmP<T> p) {
    grid_dep_sync();
    constexpr int TM = BM / 16, TN = BN / 16;
    constexpr int ITA = BM / 64;                   // float4 loads of A per thread (vector path)
    static_assert(BM == 128 || BM == 64, "row tile");
    constexpr int LDA = BM + 4, LDB = BN + 4;
    constexpr int NB4 = BK * BN / 4;               // float4 slots of a B tile
    constexpr int ITB = (NB4 + NT - 1) / NT;
    __shared__ __align__(16) float As[2][BK][LDA];
    __shared__ __align__(16) float Bs[2][BK][LDB];

    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.x * BM, j0 = blockIdx.y * BN;

    RowInfo ri[ITA];
#pragma unroll
    for (int i = 0; i < ITA; ++i) ri[i] = make_row<MODE>(p, m0 + (tid >> 2) + 64 * i);

    float ra[8], rb[ITB * 4];

    auto loadA = [&](int k0) {
        if (p.vecA) {
            const int k = k0 + (tid & 3) * 4;
            int r = 0, s = 0, c = k;
            if (!p.pointwise) { const int rs = k / p.Cs; c = k - rs * p.Cs; r = rs / p.kw; s = rs - r * p.kw; }
#pragma unroll
            for (int i = 0; i < ITA; ++i) {
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (ri[i].ok && k < p.Kg) {
                    long long off;
                    if (p.pointwise) off = (long long)(m0 + (tid >> 2) + 64 * i) * p.Cs + k;
                    else off = src_offset<MODE>(p, ri[i], r, s, c);
                    if (off >= 0) v = ldg4(p.A + off);
                }
                ra[4 * i + 0] = v.x; ra[4 * i + 1] = v.y; ra[4 * i + 2] = v.z; ra[4 * i + 3] = v.w;
            }
        } else {
            const int k = k0 + (tid & 15);
            const int rs = k / p.Cs, c = k - rs * p.Cs, r = rs / p.kw, s = rs - r * p.kw;
#pragma unroll
            for (int i = 0; i < TM; ++i) {
                float v = 0.f;
                const int m = m0 + (tid >> 4) + 16 * i;
                if (m < p.M && k < p.Kg) {
                    const RowInfo q = make_row<MODE>(p, m);
                    const long long off = src_offset<MODE>(p, q, r, s, c);
                    if (off >= 0) v = ldg1(p.A + off);
                }
                ra[i] = v;
            }
        }
    };
    auto storeA = [&](int buf) {
        if (p.vecA) {
            const int kk = (tid & 3) * 4, row = tid >> 2;
#pragma unroll
            for (int i = 0; i < ITA; ++i)
#pragma unroll
                for (int e = 0; e < 4; ++e) As[buf][kk + e][row + 64 * i] = ra[4 * i + e];
        } else {
            const int kk = tid & 15;
#pragma unroll
            for (int i = 0; i < TM; ++i) As[buf][kk][(tid >> 4) + 16 * i] = ra[i];
        }
    };
    auto loadB = [&](int k0) {
#pragma unroll
        for (int t = 0; t < ITB; ++t) {
            const int q = tid + t * NT;
            float v[4] = {0.f, 0.f, 0.f, 0.f};
            if (q < NB4) {
                if (MODE == 0) {                     // B[k][j] = W[k*Cd + j]
                    const int kk = q / (BN / 4), j = j0 + (q % (BN / 4)) * 4, k = k0 + kk;
                    if (k < p.Kg) {
                        const T* src = p.B + (long long)k * p.Cd + j;
                        if (p.vecB) {
                            if (j < p.Cd) { const float4 w = ldg4(src); v[0] = w.x; v[1] = w.y; v[2] = w.z; v[3] = w.w; }
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e) if (j + e < p.Cd) v[e] = ldg1(src + e);
                        }
                    }
                } else {                             // B[k=(rs,c)][j] = W[(rs*Cd + j)*Cs + c]
                    const int jj = q >> 2, j = j0 + jj, k = k0 + (q & 3) * 4;
                    if (j < p.Cd) {
                        if (p.vecB) {
                            if (k < p.Kg) {
                                const int rs = k / p.Cs, c = k - rs * p.Cs;
                                const float4 w = ldg4(p.B + ((long long)rs * p.Cd + j) * p.Cs + c);
                                v[0] = w.x; v[1] = w.y; v[2] = w.z; v[3] = w.w;
                            }
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const int ke = k + e;
                                if (ke < p.Kg) { const int rs = ke / p.Cs, c = ke - rs * p.Cs; v[e] = ldg1(p.B + ((long long)rs * p.Cd + j) * p.Cs + c); }
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) rb[4 * t + e] = v[e];
        }
    };
    auto storeB = [&](int buf) {
#pragma unroll
        for (int t = 0; t < ITB; ++t) {
            const int q = tid + t * NT;
            if (q < NB4) {
                if (MODE == 0) {
                    const int kk = q / (BN / 4), jq = (q % (BN / 4)) * 4;
                    *reinterpret_cast<float4*>(&Bs[buf][kk][jq]) = make_float4(rb[4 * t], rb[4 * t + 1], rb[4 * t + 2], rb[4 * t + 3]);
                } else {
                    const int jj = q >> 2, kk = (q & 3) * 4;
#pragma unroll
                    for (int e = 0; e < 4; ++e) Bs[buf][kk + e][jj] = rb[4 * t + e];
                }
            }
        }
    };

    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

    const int kt0 = blockIdx.z * p.kt_per;
    const int ktiles = min((p.Kg + BK - 1) / BK, kt0 + p.kt_per);
    loadA(kt0 * BK); loadB(kt0 * BK);
    storeA(0); storeB(0);
    __syncthreads();
    for (int kt = kt0; kt < ktiles; ++kt) {
        const int buf = (kt - kt0) & 1;
        if (kt + 1 < ktiles) { loadA((kt + 1) * BK); loadB((kt + 1) * BK); }
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[TM], b[TN];
            const float4 a0 = *reinterpret_cast<const float4*>(&As[buf][kk][ty * 4]);
            a[0] = a0.x; a[1] = a0.y; a[2] = a0.z; a[3] = a0.w;
            if constexpr (TM == 8) {
                const float4 a1 = *reinterpret_cast<const float4*>(&As[buf][kk][64 + ty * 4]);
                a[4] = a1.x; a[5] = a1.y; a[6] = a1.z; a[7] = a1.w;
            }
            if constexpr (TN == 8) {
                const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][kk][tx * 4]);
                const float4 b1 = *reinterpret_cast<const float4*>(&Bs[buf][kk][64 + tx * 4]);
                b[0] = b0.x; b[1] = b0.y; b[2] = b0.z; b[3] = b0.w; b[4] = b1.x; b[5] = b1.y; b[6] = b1.z; b[7] = b1.w;
            } else if constexpr (TN == 4) {
                const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][kk][tx * 4]);
                b[0] = b0.x; b[1] = b0.y; b[2] = b0.z; b[3] = b0.w;
            } else {
                const float2 b0 = *reinterpret_cast<const float2*>(&Bs[buf][kk][tx * 2]);
                b[0] = b0.x; b[1] = b0.y;
            }
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        if (kt + 1 < ktiles) {
            storeA(buf ^ 1); storeB(buf ^ 1);
            __syncthreads();
        }
    }

    // epilogue: bias, activation, residual-gradient addend, store (16-byte stores when aligned)
    T* const Dz = p.D + (long long)blockIdx.z * p.M * p.Cd;
    constexpr int GW = TN >= 4 ? 4 : 2;            // columns per contiguous group
    constexpr int NG = TN / GW;
    const bool vecD = p.alignD && (p.Cd % GW) == 0;
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int m = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
        if (m >= p.M) continue;
#pragma unroll
        for (int gq = 0; gq < NG; ++gq) {
            const int jc = j0 + gq * 64 + tx * GW;
            if (jc >= p.Cd) continue;
            const long long o = (long long)m * p.Cd + jc;
            float v[GW];
#pragma unroll
            for (int e = 0; e < GW; ++e) {
                float t = acc[i][gq * GW + e];
                if (p.bias && jc + e < p.Cd) t += __ldg(p.bias + jc + e);
                v[e] = apply_act(t, p.act);
            }
            if (vecD) {
                if constexpr (GW == 4) {
                    if (p.addend) { const float4 a = ldg4(p.addend + o); v[0] += a.x; v[1] += a.y; v[2] += a.z; v[3] += a.w; }
                    st4(Dz + o, v[0], v[1], v[2], v[3]);
                } else {
                    if (p.addend) { v[0] += ldg1(p.addend + o); v[1] += ldg1(p.addend + o + 1); }
                    st2(Dz + o, v[0], v[1]);
                }
            } else {
#pragma unroll
                for (int e = 0; e < GW; ++e)
                    if (jc + e < p.Cd) st1(Dz + o + e, v[e] + (p.addend ? ldg1(p.addend + o + e) : 0.f));
            }
        }
    }
}

// ---- weight gradient ---------------------------------------------------------------------------
template <typename T>
struct WgP {
    const T* X;
    const T* dY;
    float* out;            // dW, or the split partials [S][Kg][Cout]
    int M, Kg, Cout, Cs, Hs, Ws, Ho, Wo, kh, kw, stride, ph, pw;
    int chunk;             // rows of M per split (multiple of 16)
    int vecA, vecB, vecO, pointwise;
};

template <int BI, typename T>
__global__ void __launch_bounds__(NT) conv_wgrad_kernel(const WgP<T> p) {
    grid_dep_sync();
    constexpr int BJ = 64, TM = BI / 16;
    constexpr int LDA = BI + 4, LDB = BJ + 4;
    constexpr int ITA = BK * BI / 4 / NT;          // float4 loads of A per thread (2 or 1)
    __shared__ __align__(16) float As[2][BK][LDA];
    __shared__ __align__(16) float Bs[2][BK][LDB];

    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int i0 = blockIdx.x * BI, j0 = blockIdx.y * BJ;
    const int mbeg = blockIdx.z * p.chunk;
    const int mend = min(p.M, mbeg + p.chunk);
    const int howo = p.Ho * p.Wo;

    // this thread's fixed reduction-operand column (k) and its tap
    const int kA = p.vecA ? i0 + (tid % (BI / 4)) * 4 : i0 + (tid % BI);
    int rA = 0, sA = 0, cA = kA;
    if (!p.pointwise) { const int rs = kA / p.Cs; cA = kA - rs * p.Cs; rA = rs / p.kw; sA = rs - rA * p.kw; }

    auto x_offset = [&](int m) -> long long {
        if (p.pointwise) return (long long)m * p.Cs + kA;
        const int n = m / howo, rem = m - n * howo, ho = rem / p.Wo, wo = rem - ho * p.Wo;
        const int hs = ho * p.stride - p.ph + rA, ws = wo * p.stride - p.pw + sA;
        if (hs < 0 || hs >= p.Hs || ws < 0 || ws >= p.Ws) return -1;
        return ((long long)((n * p.Hs + hs) * p.Ws + ws)) * p.Cs + cA;
    };

    float ra[8], rb[4];
    auto loadA = [&](int mrow0) {
        if (p.vecA) {
#pragma unroll
            for (int t = 0; t < ITA; ++t) {
                const int m = mrow0 + tid / (BI / 4) + t * (NT / (BI / 4));
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (m < mend && kA < p.Kg) { const long long off = x_offset(m); if (off >= 0) v = ldg4(p.X + off); }
                ra[4 * t] = v.x; ra[4 * t + 1] = v.y; ra[4 * t + 2] = v.z; ra[4 * t + 3] = v.w;
            }
        } else {
#pragma unroll
            for (int t = 0; t < BI / 16; ++t) {
                const int m = mrow0 + tid / BI + t * (NT / BI);
                float v = 0.f;
                if (m < mend && kA < p.Kg) { const long long off = x_offset(m); if (off >= 0) v = ldg1(p.X + off); }
                ra[t] = v;
            }
        }
    };
    auto storeA = [&](int buf) {
        if (p.vecA) {
#pragma unroll
            for (int t = 0; t < ITA; ++t)
                *reinterpret_cast<float4*>(&As[buf][tid / (BI / 4) + t * (NT / (BI / 4))][(tid % (BI / 4)) * 4]) =
                    make_float4(ra[4 * t], ra[4 * t + 1], ra[4 * t + 2], ra[4 * t + 3]);
        } else {
#pragma unroll
            for (int t = 0; t < BI / 16; ++t) As[buf][tid / BI + t * (NT / BI)][tid % BI] = ra[t];
        }
    };
    auto loadB = [&](int mrow0) {
        if (p.vecB) {
            const int m = mrow0 + (tid >> 4), j = j0 + (tid & 15) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (m < mend && j < p.Cout) v = ldg4(p.dY + (long long)m * p.Cout + j);
            rb[0] = v.x; rb[1] = v.y; rb[2] = v.z; rb[3] = v.w;
        } else {
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int m = mrow0 + (tid >> 6) + t * 4, j = j0 + (tid & 63);
                rb[t] = (m < mend && j < p.Cout) ? ldg1(p.dY + (long long)m * p.Cout + j) : 0.f;
            }
        }
    };
    auto storeB = [&](int buf) {
        if (p.vecB) *reinterpret_cast<float4*>(&Bs[buf][tid >> 4][(tid & 15) * 4]) = make_float4(rb[0], rb[1], rb[2], rb[3]);
        else {
#pragma unroll
            for (int t = 0; t < 4; ++t) Bs[buf][(tid >> 6) + t * 4][tid & 63] = rb[t];
        }
    };

    float acc[TM][4];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    const int steps = (mend - mbeg + BK - 1) / BK;
    if (steps > 0) {
        loadA(mbeg); loadB(mbeg);
        storeA(0); storeB(0);
        __syncthreads();
    }
    for (int st = 0; st < steps; ++st) {
        const int buf = st & 1;
        if (st + 1 < steps) { loadA(mbeg + (st + 1) * BK); loadB(mbeg + (st + 1) * BK); }
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[TM];
            const float4 a0 = *reinterpret_cast<const float4*>(&As[buf][kk][ty * 4]);
            a[0] = a0.x; a[1] = a0.y; a[2] = a0.z; a[3] = a0.w;
            if constexpr (TM == 8) {
                const float4 a1 = *reinterpret_cast<const float4*>(&As[buf][kk][64 + ty * 4]);
                a[4] = a1.x; a[5] = a1.y; a[6] = a1.z; a[7] = a1.w;
            }
            const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][kk][tx * 4]);
            const float b[4] = {b0.x, b0.y, b0.z, b0.w};
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        if (st + 1 < steps) {
            storeA(buf ^ 1); storeB(buf ^ 1);
            __syncthreads();
        }
    }
    float* out = p.out + (long long)blockIdx.z * p.Kg * p.Cout;
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int k = i0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
        if (k >= p.Kg) continue;
        const int jc = j0 + tx * 4;
        if (p.vecO) {
            if (jc < p.Cout) *reinterpret_cast<float4*>(out + (long long)k * p.Cout + jc) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (jc + j < p.Cout) out[(long long)k * p.Cout + jc + j] = acc[i][j];
        }
    }
}

// out[e] = sum_z partial[z][e]: the fixed-order second pass of every split reduction.  Block (32, 8): eight
// interleaved runs over z per element (two loads in flight each), combined in run order through shared memory.
__global__ void __launch_bounds__(256) split_reduce_kernel(const float* __restrict__ partial, int S, long long count, float* __restrict__ out) {
    grid_dep_sync();
    __shared__ float sh[8][33];
    const long long e = (long long)blockIdx.x * 32 + threadIdx.x;
    float s0 = 0.f, s1 = 0.f;
    if (e < count)
        for (int z = threadIdx.y; z < S; z += 16) {
            const float a = partial[(long long)z * count + e];
            const float b = z + 8 < S ? partial[(long long)(z + 8) * count + e] : 0.f;
            s0 += a; s1 += b;
        }
    sh[threadIdx.y][threadIdx.x] = s0 + s1;
    __syncthreads();
    if (threadIdx.y == 0 && e < count) {
        float s = 0.f;
#pragma unroll
        for (int y = 0; y < 8; ++y) s += sh[y][threadIdx.x];
        out[e] = s;
    }
}

// the same for few slices: one thread per element, z ascending
__global__ void __launch_bounds__(256) split_reduce_flat_kernel(const float* __restrict__ partial, int S, long long count, float* __restrict__ out) {
    grid_dep_sync();
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= count) return;
    float s = 0.f;
    for (int z = 0; z < S; ++z) s += partial[(long long)z * count + e];
    out[e] = s;
}

static inline void launch_split_reduce(const float* partial, int S, long long count, float* out, cudaStream_t st) {
    if (S >= 16) launch(split_reduce_kernel, dim3((unsigned)((count + 31) / 32)), dim3(32, 8), 0, st, partial, S, count, out);
    else launch(split_reduce_flat_kernel, dim3((unsigned)((count + 255) / 256)), dim3(256), 0, st, partial, S, count, out);
}

// out[e] = sum_z partial[z][e] (+ bias[column]) (+ addend[e]), z ascending
__global__ void split_reduce_add_kernel(const float* __restrict__ partial, int S, long long count4, const float* __restrict__ addend,
                                        const float* __restrict__ bias, int Cd, float* __restrict__ out) {
    grid_dep_sync();
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= count4) return;
    float4 s = __ldg(reinterpret_cast<const float4*>(partial) + e);
    for (int z = 1; z < S; ++z) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(partial) + (long long)z * count4 + e);
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    if (bias) {
        const int c = (int)((e * 4) % Cd);
        s.x += __ldg(bias + c); s.y += __ldg(bias + (c + 1) % Cd); s.z += __ldg(bias + (c + 2) % Cd); s.w += __ldg(bias + (c + 3) % Cd);
    }
    if (addend) { const float4 a = __ldg(reinterpret_cast<const float4*>(addend) + e); s.x += a.x; s.y += a.y; s.z += a.z; s.w += a.w; }
    reinterpret_cast<float4*>(out)[e] = s;
}

struct WgPlan { int BI, S, chunk; };

WgPlan plan_wgrad(const ConvGeom& g) {
    const long long M = (long long)g.N * g.Ho * g.Wo;
    const int Kg = g.kh * g.kw * g.Cin;
    WgPlan w;
    w.BI = Kg > 64 ? 128 : 64;
    const int tiles = ((Kg + w.BI - 1) / w.BI) * ((g.Cout + 63) / 64);
    long long S = (4LL * sm_count() + tiles - 1) / tiles;          // ~4 resident blocks per SM hide the load latency
    long long maxS = (M + 255) / 256;
    const long long cap = (4LL << 20) / ((long long)Kg * g.Cout);  // keep the partials within 4 Mi floats
    if (maxS > cap) maxS = cap;
    if (S > maxS) S = maxS;
    if (S < 1) S = 1;
    long long chunk = (M + S - 1) / S;
    chunk = (chunk + BK - 1) / BK * BK;
    w.chunk = (int)chunk;
    w.S = (int)((M + chunk - 1) / chunk);
    return w;
}

// Tile shapes: (rows, columns, relative efficiency of the register micro-tile, resident blocks per SM).
struct TileOpt { int bm, bn; float eff; int slots; };
constexpr TileOpt kTiles[] = {{128, 128, 1.00f, 2}, {128, 64, 0.85f, 3}, {64, 128, 0.85f, 3}, {64, 64, 0.65f, 4},
                              {128, 32, 0.55f, 4}, {64, 32, 0.45f, 6}};

// Estimated cost of covering an M x N output: full waves of resident blocks, each block slowed by its
// co-residents, padding included through the tile counts.
inline int pick_tile(long long M, int N) {
    const long long sms = sm_count();
    int best = 0;
    double best_t = 1e300;
    for (int i = 0; i < (int)(sizeof(kTiles) / sizeof(kTiles[0])); ++i) {
        const TileOpt& t = kTiles[i];
        const long long tiles = ((M + t.bm - 1) / t.bm) * ((N + t.bn - 1) / t.bn);
        const long long waves = (tiles + sms * t.slots - 1) / (sms * t.slots);
        const double cost = (double)waves * t.slots * t.bm * t.bn / t.eff;
        if (cost < best_t) { best_t = cost; best = i; }
    }
    return best;
}

// Split of the reduction dimension for outputs too small to fill the GPU (late layers: few pixels, many
// channels).  Only plain products qualify (no bias, no activation); the addend joins in the second pass.
struct GemmPlan { int tile, S, kt_per; };
inline GemmPlan plan_gemm(long long M, int N, int Kg, bool plain) {
    GemmPlan gp;
    gp.tile = pick_tile(M, N);
    const TileOpt& t = kTiles[gp.tile];
    const long long tiles = ((M + t.bm - 1) / t.bm) * ((N + t.bn - 1) / t.bn);
    const int ktiles = (Kg + BK - 1) / BK;
    long long S = 1;
    if (plain && tiles < 2LL * sm_count() && ktiles >= 8 && (M * N) % 4 == 0) {
        S = (3LL * sm_count() + tiles - 1) / tiles;
        if (S > ktiles / 4) S = ktiles / 4;
        if (S > 16) S = 16;
        if (S < 1) S = 1;
    }
    gp.kt_per = (int)((ktiles + S - 1) / S);
    gp.S = (ktiles + gp.kt_per - 1) / gp.kt_per;
    return gp;
}

template <int MODE, typename T>
void launch_conv_gemm(GemmP<T> p, float* scratch, cudaStream_t st) {
    constexpr bool kF32 = sizeof(T) == 4;
    const bool plain = kF32 && p.act == 0 && scratch != nullptr && (reinterpret_cast<uintptr_t>(p.D) & 15) == 0 &&
                       (reinterpret_cast<uintptr_t>(p.addend) & 15) == 0;
    const GemmPlan gp = plan_gemm(p.M, p.Cd, p.Kg, plain);
    const TileOpt t = kTiles[gp.tile];
    const dim3 grid((p.M + t.bm - 1) / t.bm, (p.Cd + t.bn - 1) / t.bn, gp.S);
    T* const out = p.D;
    const T* const addend = p.addend;
    const float* const bias = p.bias;
    p.kt_per = gp.kt_per;
    if (gp.S > 1) { p.D = reinterpret_cast<T*>(scratch); p.addend = nullptr; p.bias = nullptr; p.alignD = 1; }
#define FTP_LAUNCH(BM_, BN_) if (t.bm == BM_ && t.bn == BN_) launch(conv_gemm_kernel<BM_, BN_, MODE, T>, grid, dim3(NT), 0, st, p);
    FTP_LAUNCH(128, 128) FTP_LAUNCH(128, 64) FTP_LAUNCH(64, 128) FTP_LAUNCH(64, 64) FTP_LAUNCH(128, 32) FTP_LAUNCH(64, 32)
#undef FTP_LAUNCH
    if constexpr (kF32) {
        if (gp.S > 1) {
            const long long count4 = (long long)p.M * p.Cd / 4;
            launch(split_reduce_add_kernel, dim3((unsigned)((count4 + 255) / 256)), dim3(256), 0, st, scratch, gp.S, count4, reinterpret_cast<const float*>(addend), bias, p.Cd,
                                                                                      reinterpret_cast<float*>(out));
        }
    }
}

inline bool a16(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; }
inline bool is_pointwise(const ConvGeom& g) { return g.kh == 1 && g.kw == 1 && g.stride == 1 && g.ph == 0 && g.pw == 0; }

}  // namespace

size_t conv_gemm_scratch_floats(const ConvGeom& g) {
    const long long Mf = (long long)g.N * g.Ho * g.Wo, Mb = (long long)g.N * g.H * g.W;
    const GemmPlan f = plan_gemm(Mf, g.Cout, g.kh * g.kw * g.Cin, true), b = plan_gemm(Mb, g.Cin, g.kh * g.kw * g.Cout, true);
    const size_t nf = f.S > 1 ? (size_t)f.S * Mf * g.Cout : 0, nb = b.S > 1 ? (size_t)b.S * Mb * g.Cin : 0;
    return nf > nb ? nf : nb;
}

namespace {
constexpr int kVec = 4;     // elements per vector access in these kernels (16 bytes of float, 8 of bfloat16)
template <typename T> inline bool avec(const void* q) { return (reinterpret_cast<uintptr_t>(q) & (kVec * sizeof(T) - 1)) == 0; }

template <typename T>
void conv_fwd_t(const T* x, const T* w, const float* bias, T* y, float* scratch, const ConvGeom& g, int act, cudaStream_t st) {
    GemmP<T> p{};
    p.A = x; p.B = w; p.bias = bias; p.addend = nullptr; p.D = y;
    p.M = g.N * g.Ho * g.Wo; p.Kg = g.kh * g.kw * g.Cin; p.Cd = g.Cout;
    p.Hs = g.H; p.Ws = g.W; p.Cs = g.Cin; p.Hd = g.Ho; p.Wd = g.Wo;
    p.kh = g.kh; p.kw = g.kw; p.stride = g.stride; p.ph = g.ph; p.pw = g.pw;
    p.act = act; p.vecA = (g.Cin % 4 == 0) && avec<T>(x); p.vecB = (g.Cout % 4 == 0) && avec<T>(w); p.alignD = avec<T>(y);
    p.pointwise = is_pointwise(g);
    launch_conv_gemm<0, T>(p, scratch, st);
}

template <typename T>
void conv_dgrad_t(const T* dy, const T* w, const T* addend, T* dx, float* scratch, const ConvGeom& g, cudaStream_t st) {
    GemmP<T> p{};
    p.A = dy; p.B = w; p.bias = nullptr; p.addend = addend; p.D = dx;
    p.M = g.N * g.H * g.W; p.Kg = g.kh * g.kw * g.Cout; p.Cd = g.Cin;
    p.Hs = g.Ho; p.Ws = g.Wo; p.Cs = g.Cout; p.Hd = g.H; p.Wd = g.W;
    p.kh = g.kh; p.kw = g.kw; p.stride = g.stride; p.ph = g.ph; p.pw = g.pw;
    p.act = 0; p.vecA = (g.Cout % 4 == 0) && avec<T>(dy); p.vecB = (g.Cout % 4 == 0) && avec<T>(w); p.alignD = avec<T>(dx) && avec<T>(addend);
    p.pointwise = is_pointwise(g);
    launch_conv_gemm<1, T>(p, scratch, st);
}

template <typename T>
void conv_wgrad_t(const T* x, const T* dy, float* dw, float* scratch, const ConvGeom& g, cudaStream_t st) {
    const WgPlan w = plan_wgrad(g);
    WgP<T> p{};
    p.X = x; p.dY = dy; p.out = w.S > 1 ? scratch : dw;
    p.M = g.N * g.Ho * g.Wo; p.Kg = g.kh * g.kw * g.Cin; p.Cout = g.Cout; p.Cs = g.Cin; p.Hs = g.H; p.Ws = g.W;
    p.Ho = g.Ho; p.Wo = g.Wo; p.kh = g.kh; p.kw = g.kw; p.stride = g.stride; p.ph = g.ph; p.pw = g.pw;
    p.chunk = w.chunk; p.vecA = (g.Cin % 4 == 0) && avec<T>(x); p.vecB = (g.Cout % 4 == 0) && avec<T>(dy);
    p.vecO = (g.Cout % 4 == 0) && a16(p.out) && ((long long)p.Kg * g.Cout) % 4 == 0; p.pointwise = is_pointwise(g);
    const dim3 grid((p.Kg + w.BI - 1) / w.BI, (g.Cout + 63) / 64, w.S);
    if (w.BI == 128) launch(conv_wgrad_kernel<128, T>, grid, dim3(NT), 0, st, p);
    else launch(conv_wgrad_kernel<64, T>, grid, dim3(NT), 0, st, p);
    if (w.S > 1) {
        const long long count = (long long)p.Kg * g.Cout;
        launch_split_reduce(scratch, w.S, count, dw, st);
    }
}
}  // namespace

void conv_fwd_f32(const float* x, const float* w, const float* bias, float* y, float* scratch, const ConvGeom& g, int act, cudaStream_t st) {
    conv_fwd_t<float>(x, w, bias, y, scratch, g, act, st);
}
void conv_dgrad_f32(const float* dy, const float* w, const float* addend, float* dx, float* scratch, const ConvGeom& g, cudaStream_t st) {
    conv_dgrad_t<float>(dy, w, addend, dx, scratch, g, st);
}
void conv_fwd_bf16_simt(const __nv_bfloat16* x, const __nv_bfloat16* w, const float* bias, __nv_bfloat16* y, const ConvGeom& g, int act, cudaStream_t st) {
    conv_fwd_t<__nv_bfloat16>(x, w, bias, y, nullptr, g, act, st);
}
void conv_dgrad_bf16_simt(const __nv_bfloat16* dy, const __nv_bfloat16* w, const __nv_bfloat16* addend, __nv_bfloat16* dx, const ConvGeom& g, cudaStream_t st) {
    conv_dgrad_t<__nv_bfloat16>(dy, w, addend, dx, nullptr, g, st);
}

void split_reduce_f32(const float* partial, int S, long long count, float* out, cudaStream_t st) {
    launch_split_reduce(partial, S, count, out, st);
}

size_t conv_wgrad_scratch_floats(const ConvGeom& g) {
    const WgPlan w = plan_wgrad(g);
    return w.S > 1 ? (size_t)w.S * g.kh * g.kw * g.Cin * g.Cout : 0;
}

void conv_wgrad_f32(const float* x, const float* dy, float* dw, float* scratch, const ConvGeom& g, cudaStream_t st) {
    conv_wgrad_t<float>(x, dy, dw, scratch, g, st);
}
void conv_wgrad_bf16_simt(const __nv_bfloat16* x, const __nv_bfloat16* dy, float* dw, float* scratch, const ConvGeom& g, cudaStream_t st) {
    conv_wgrad_t<__nv_bfloat16>(x, dy, dw, scratch, g, st);
}

}  // namespace ftp
