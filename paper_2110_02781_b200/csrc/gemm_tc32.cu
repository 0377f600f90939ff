// float contractions on the tensor cores with float-level accuracy: every operand x is split into
// hi = x with the low 13 mantissa bits cleared (exactly representable as tf32) and lo = x - hi (exact), and
// the product is accumulated as hi*hi + hi*lo + lo*hi with tcgen05.mma kind::tf32 into a float accumulator in
// tensor memory.  The dropped lo*lo term and the tf32 truncation of lo are below 2^-20 relative, which keeps
// the float path within 1e-4 of a float64 reference while the math leaves the SIMT pipes.  The tensor core
// reads only the upper 19 bits of a tf32 operand, so a float tile as it lies in memory already is its hi part.
//
// Two kernels, one 128 x BN tile (and one slice of the reduction) per CTA, warp roles as in the bf16 kernels:
//  * tc32_kernel: both operands with the reduction contiguous (forward with pre-transposed weights, data
//    gradient).  Warp 0 streams 128 x 32 and BN x 32 float tiles with TMA (128-byte swizzle, zero fill); warps
//    2-5 write the lo tile of A (and of B, unless the caller keeps B's lo part in memory, as the model does for
//    its weights), make the writes visible to the tensor-core proxy and signal warp 1, which issues the 3 x 4
//    MMAs (K = 8) of the stage; at the end warps 2-5 read the accumulator, stage it in shared memory and store
//    it with TMA.
//  * tc32_wgrad_kernel: both operands have the reduction as their slow dimension (activations and output
//    gradients of the weight gradient); the tensor core takes them as they land (MN-major operands), and the
//    converter warps only add the lo parts.
// Every wait is bounded; see gemm_tc.cu for the error protocol.
#include <cstdlib>
#include "gemm_tc_common.cuh"
#include "bn_math.cuh"

namespace ftp {
using namespace tc;
namespace {

constexpr int T32_BK = 32;          // floats per 128-byte row

__device__ __forceinline__ void mbar_arrive(uint32_t bar) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory"); }

__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}"
                 ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// The tensor core reads only the upper 19 bits of a tf32 operand, so the tile as TMA delivered it already is the
// "hi" part; the "lo" part x - trunc(x) goes to the buffer `lo_off` bytes further.  Elementwise, so the swizzled
// placement does not matter.  `threads` cooperating threads, `t` this thread's rank.
__device__ __forceinline__ void split_tile(const uint8_t* hi, uint8_t* lo, int bytes, int t, int threads) {
    for (int i = t * 16; i < bytes; i += threads * 16) {
        const float4 v = *reinterpret_cast<const float4*>(hi + i);
        float4 l;
        l.x = v.x - __uint_as_float(__float_as_uint(v.x) & 0xffffe000u);
        l.y = v.y - __uint_as_float(__float_as_uint(v.y) & 0xffffe000u);
        l.z = v.z - __uint_as_float(__float_as_uint(v.z) & 0xffffe000u);
        l.w = v.w - __uint_as_float(__float_as_uint(v.w) & 0xffffe000u);
        *reinterpret_cast<float4*>(lo + i) = l;
    }
}

__device__ __forceinline__ float tf32_lo_of(float v) { return v - __uint_as_float(__float_as_uint(v) & 0xffffe000u); }

// Batch norm + activation on a float4 of four consecutive channels (constants in registers), zero where !keep
struct Xf4 {
    float4 mu, sc, of;
    __device__ __forceinline__ void load(const BnXform& x, int c, bool ok) {
        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        mu = ok ? __ldg(reinterpret_cast<const float4*>(x.mean + c)) : z;
        sc = ok ? __ldg(reinterpret_cast<const float4*>(x.scale + c)) : z;
        of = ok ? __ldg(reinterpret_cast<const float4*>(x.offset + c)) : z;
    }
    __device__ __forceinline__ float4 apply(float4 v, float lo, float hi, bool keep) const {
        float4 o;
        o.x = keep ? xf_z(v.x, mu.x, sc.x, of.x, lo, hi) : 0.f;
        o.y = keep ? xf_z(v.y, mu.y, sc.y, of.y, lo, hi) : 0.f;
        o.z = keep ? xf_z(v.z, mu.z, sc.z, of.z, lo, hi) : 0.f;
        o.w = keep ? xf_z(v.w, mu.w, sc.w, of.w, lo, hi) : 0.f;
        return o;
    }
};

// A K-major 128 x 32 float tile (128-byte rows, 16-byte pieces XOR-swizzled with row % 8) whose values are the input
// of a batch norm: 128 threads replace every value by its normalised, activated value (rows past `rows_valid` and
// channels past the end of the reduction become zero, as padding must) and write the lo part.  Thread t owns the
// physical piece t % 8 of rows t / 8 + 16 j, which is the same logical piece -- the same four channels -- in every row.
__device__ __forceinline__ void xform_split_tile_k(uint8_t* hi, uint8_t* lo, int t, const Xf4& c, float zlo, float zhi, bool chan_ok, int rows_valid) {
    const int row0 = t >> 3;
    uint8_t* p = hi + row0 * 128 + (t & 7) * 16;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int row = row0 + 16 * j;
        const float4 v = *reinterpret_cast<const float4*>(p + j * 2048);
        const float4 z = c.apply(v, zlo, zhi, chan_ok && row < rows_valid);
        *reinterpret_cast<float4*>(p + j * 2048) = z;
        *reinterpret_cast<float4*>(p + j * 2048 + (lo - hi)) = make_float4(tf32_lo_of(z.x), tf32_lo_of(z.y), tf32_lo_of(z.z), tf32_lo_of(z.w));
    }
}

// The same for an MN-major operand of the weight gradient: `slabs` slabs of 32 reduction rows x 32 channels (128-byte
// rows, 32-byte pieces XOR-swizzled with row % 4), 256 threads.  Thread t owns the 16-byte piece t % 8 of row t / 8 in
// every slab: channels 8 * ((t % 8 / 2) ^ (row % 4)) + 4 * (t % 2) of the slab, whose constants are c[slab].
__device__ __forceinline__ void xform_split_slabs_mn(uint8_t* hi, uint8_t* lo, int slabs, int t, const Xf4 (&c)[4], const bool (&chan_ok)[4], float zlo,
                                                     float zhi, bool row_ok) {
#pragma unroll
    for (int n = 0; n < 4; ++n) {
        if (n < slabs) {
            uint8_t* q = hi + n * 4096 + t * 16;
            const float4 v = *reinterpret_cast<const float4*>(q);
            const float4 z = c[n].apply(v, zlo, zhi, row_ok && chan_ok[n]);
            *reinterpret_cast<float4*>(q) = z;
            *reinterpret_cast<float4*>(q + (lo - hi)) = make_float4(tf32_lo_of(z.x), tf32_lo_of(z.y), tf32_lo_of(z.z), tf32_lo_of(z.w));
        }
    }
}

struct T32Params {
    float* D;              // output [S][M][N]: the result itself when S == 1, else partial sums over slices of the reduction
    const float* addend;   // gemm with S == 1 only, nullable
    int M, N, K;           // gemm: D[M,N] = A[M,K] B[N,K]^T.  wgrad: Mo = M, No = N, K = reduction rows R
    int rows_per_split;    // reduction elements per slice (a multiple of 32)
    int b_lo_given;        // gemm: the lo part of B comes from memory (mapBlo) instead of being computed per tile
    int* err;
    double* stats;         // gemm with S == 1 only, nullable: [row tiles][2][N] column sums and sums of squares of each output tile
    BnXform xf;            // xf.scale != nullptr: a batch norm applied to one operand while its tiles are split (gemm: A; wgrad: see xf_operand)
    int xf_operand;        // wgrad: 1 = the A operand is transformed, 2 = the B operand
};

// Epilogue shared by both kernels, run by warps 2..5: accumulator -> shared-memory tiles of 128 rows x 32 columns
// (the operand buffers are free by now) -> one TMA store per tile, which writes whole lines and clips at the
// edges of the output.  `have`: the accumulator is complete (or there was nothing to accumulate).
template <int BN>
__device__ __forceinline__ void epilogue32(uint8_t* smem, uint32_t tmem, const CUtensorMap* mapD, const T32Params& p, const float* addend, int m0, int n0,
                                           int split, int num_kb, bool have) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, q = warp & 3;
    if (have) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int row = q * 32 + lane, m = m0 + row;
        const float* arow = (addend && m < p.M) ? addend + (long long)m * p.N : nullptr;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
            uint32_t r[32];
            if (num_kb > 0) tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32), r);
            else {
#pragma unroll
                for (int e = 0; e < 32; ++e) r[e] = 0u;
            }
            const int nb = n0 + c * 32;
            uint8_t* trow = smem + c * (TC_BM * 128) + row * 128;
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                float4 v = make_float4(__uint_as_float(r[g * 4]), __uint_as_float(r[g * 4 + 1]), __uint_as_float(r[g * 4 + 2]), __uint_as_float(r[g * 4 + 3]));
                if (arow && nb + g * 4 < p.N) { const float4 a = __ldg(reinterpret_cast<const float4*>(arow + nb + g * 4)); v.x += a.x; v.y += a.y; v.z += a.z; v.w += a.w; }
                *reinterpret_cast<float4*>(trow + ((g ^ (row & 7)) << 4)) = v;
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");                      // the four epilogue warps
    if (have && threadIdx.x == 64) {
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c)
            if (n0 + c * 32 < p.N)
                asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
                             ::"l"(mapD), "r"(n0 + c * 32), "r"(m0), "r"(split), "r"(smem_u32(smem + c * (TC_BM * 128))) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
    if (p.stats) {
        // Column sums of the staged tile for the batch norm that follows: thread t takes column t % BN and the
        // rows of group t / BN, in double; the 128 / BN groups are added in group order.  Rows past M hold zeros.
        constexpr int G = TC_BM / BN, RPG = TC_BM / G;
        __shared__ double red[2][TC_BM];
        const int t = threadIdx.x - 64, col = t % BN, grp = t / BN;
        double s = 0.0, q = 0.0;
        if (have) {
            const uint8_t* base = smem + (col >> 5) * (TC_BM * 128) + ((col & 3) << 2);
            const int g = (col & 31) >> 2;
#pragma unroll 8
            for (int r = grp * RPG; r < (grp + 1) * RPG; ++r) {
                const double v = (double)*reinterpret_cast<const float*>(base + r * 128 + ((g ^ (r & 7)) << 4));
                s += v;
                q = fma(v, v, q);
            }
        }
        if (G > 1) {
            red[0][t] = s; red[1][t] = q;
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (grp == 0)
                for (int k = 1; k < G; ++k) { s += red[0][k * BN + col]; q += red[1][k * BN + col]; }
        }
        if (have && grp == 0 && n0 + col < p.N) {
            double* dst = p.stats + ((long long)blockIdx.y * 2) * p.N + n0 + col;
            dst[0] = s;
            dst[p.N] = q;
        }
    }
    if (have && threadIdx.x == 64) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // shared memory may be released after this
}

// twelve tf32 MMAs per 32-wide block of the reduction: hi*hi, hi*lo, lo*hi for each of its four 8-wide steps
template <int BN>
__device__ __forceinline__ void mma_block32(uint32_t tmem, uint32_t a_hi, uint32_t a_lo, uint32_t b_hi, uint32_t b_lo, bool first) {
    constexpr uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
    const uint64_t ah = umma_desc_k_sw128(a_hi), al = umma_desc_k_sw128(a_lo);
    const uint64_t bh = umma_desc_k_sw128(b_hi), bl = umma_desc_k_sw128(b_lo);
#pragma unroll
    for (int k = 0; k < T32_BK / 8; ++k) {                 // 8 reduction steps = 32 bytes further along the row
        const uint64_t o = (uint64_t)(k * 2);
        umma_tf32(tmem, ah + o, bh + o, idesc, (!first || k > 0) ? 1u : 0u);
        umma_tf32(tmem, ah + o, bl + o, idesc, 1u);
        umma_tf32(tmem, al + o, bh + o, idesc, 1u);
    }
}

// D[M,N] (one slice of the reduction per blockIdx.z) = A[M,K] B[N,K]^T, both operands with K contiguous.
// Stage: [A as loaded = hi][A lo][B hi][B lo].
template <int BN, int STAGES>
__global__ void __launch_bounds__(TC_THREADS) tc32_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                                                          const __grid_constant__ CUtensorMap mapBlo, const __grid_constant__ CUtensorMap mapD,
                                                          const T32Params p) {
    constexpr uint32_t A_BYTES = TC_BM * T32_BK * 4, B_BYTES = BN * T32_BK * 4;          // one precision part
    constexpr uint32_t STAGE_BYTES = 2 * (A_BYTES + B_BYTES);
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ __align__(8) unsigned long long bars[3 * STAGES + 1];
    __shared__ uint32_t tmem_base;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * BN, m0 = blockIdx.y * TC_BM, split = blockIdx.z;
    const int kbeg = split * p.rows_per_split, kend = min(p.K, kbeg + p.rows_per_split);
    const int num_kb = (kend - kbeg + T32_BK - 1) / T32_BK;
    const bool b_pre = p.b_lo_given != 0;
    const uint32_t tx_bytes = A_BYTES + B_BYTES + (b_pre ? B_BYTES : 0);
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[STAGES]), ready0 = smem_u32(&bars[2 * STAGES]), accum = smem_u32(&bars[3 * STAGES]);

    if (threadIdx.x == 0) {
        tma_prefetch_map(&mapA); tma_prefetch_map(&mapB); tma_prefetch_map(&mapBlo); tma_prefetch_map(&mapD);
        for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); mbar_init(ready0 + 8 * s, 128); }
        mbar_init(accum, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base)), "r"((uint32_t)BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_base;
    grid_dep_sync();                 // everything above overlaps the tail of the preceding kernel

    if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % STAGES;
                const uint32_t ph = (kb / STAGES) & 1;
                if (kb >= STAGES && !mbar_wait(empty0 + 8 * s, ph ^ 1, p.err, 11)) break;
                const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + 2 * A_BYTES;
                const int k = kbeg + kb * T32_BK;
                mbar_expect_tx(full0 + 8 * s, tx_bytes);
                tma_load_2d(sa, &mapA, k, m0, full0 + 8 * s);
                tma_load_2d(sb, &mapB, k, n0, full0 + 8 * s);
                if (b_pre) tma_load_2d(sb + B_BYTES, &mapBlo, k, n0, full0 + 8 * s);
                issued = kb + 1;
            }
            if (*((volatile int*)p.err) != 0) {
                for (int kb = max(0, issued - STAGES); kb < issued; ++kb) {
                    const unsigned long long t0 = gtime();
                    while (!mbar_test(full0 + 8 * (kb % STAGES), (kb / STAGES) & 1) && gtime() - t0 < 1000000ull) __nanosleep(128);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            bool ok = true;
            for (int kb = 0; kb < num_kb && ok; ++kb) {
                const int s = kb % STAGES;
                const uint32_t ph = (kb / STAGES) & 1;
                ok = mbar_wait(ready0 + 8 * s, ph, p.err, 12);                   // lo parts written and visible
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + 2 * A_BYTES;
                mma_block32<BN>(tmem, sa, sa + A_BYTES, sb, sb + B_BYTES, kb == 0);
                umma_commit(empty0 + 8 * s);
            }
            if (ok) umma_commit(accum);
        }
    } else {
        // ---- warps 2..5: lo part of every landed stage, then the epilogue ----
        const int t = threadIdx.x - 64;
        bool ok = true;
        const bool xf = p.xf.scale != nullptr;
        const int xf_piece = (t & 7) ^ ((t >> 3) & 7);          // logical 16-byte piece (four channels) of this thread's pieces
        for (int kb = 0; kb < num_kb && ok; ++kb) {
            const int s = kb % STAGES;
            const uint32_t ph = (kb / STAGES) & 1;
            Xf4 xc;
            const int xch = kbeg + kb * T32_BK + 4 * xf_piece;
            if (xf) xc.load(p.xf, xch, xch < p.K);               // fetched while the tile is still in flight
            ok = mbar_wait(full0 + 8 * s, ph, p.err, 13);
            if (!ok) break;
            uint8_t* st = smem + s * STAGE_BYTES;
            if (xf) xform_split_tile_k(st, st + A_BYTES, t, xc, p.xf.lo, p.xf.hi, xch < p.K, p.M - m0);
            else split_tile(st, st + A_BYTES, A_BYTES, t, 128);
            if (!b_pre) split_tile(st + 2 * A_BYTES, st + 2 * A_BYTES + B_BYTES, B_BYTES, t, 128);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // generic-proxy writes -> visible to the tensor cores
            mbar_arrive(ready0 + 8 * s);
        }
        const bool have = ok && (num_kb > 0 ? mbar_wait(accum, 0, p.err, 14) : true);
        epilogue32<BN>(smem, tmem, &mapD, p, p.addend, m0, n0, split, num_kb, have);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)BN) : "memory");
}

// Weight gradient: partials [slice][Mo][No] of X[R][Mo]^T dY[R][No].  Both operands have the reduction (rows) as
// their slow dimension, so they are fed to the tensor core as they lie: a TMA box of 32 reduction rows x 32
// columns with the 128-byte swizzle is four groups of 8 rows x 128 bytes, which is the MN-major operand layout of
// the tensor core (one group per 8-deep MMA; 32-column slabs side by side, one slab = 4096 bytes apart).  A stage
// is [A hi = as loaded][A lo][B hi = as loaded][B lo]; the converter warps only write the lo parts.
template <int BN> struct Wg32Smem {
    static constexpr uint32_t A_BYTES = TC_BM * T32_BK * 4, B_BYTES = BN * T32_BK * 4;
    static constexpr uint32_t STAGE_BYTES = 2 * (A_BYTES + B_BYTES);
    static constexpr int NSTG_FIT = (226 * 1024) / (int)STAGE_BYTES;
    static constexpr int NSTG = BN <= 64 ? 2 : (NSTG_FIT > 5 ? 5 : NSTG_FIT);
    static constexpr int TOTAL = NSTG * (int)STAGE_BYTES + 1024;
};

// MN-major operand of 32-bit elements: 128-byte swizzle with 32-byte atoms (the 32-byte piece index of a 128-byte row is
// XORed with row % 4), groups of 4 reduction rows 512 bytes apart, runs of 32 columns `slab_bytes` apart
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t saddr, uint32_t slab_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFF);          // start address
    d |= (uint64_t)(slab_bytes >> 4) << 16;          // leading byte offset: from one 128-byte run of columns to the next
    d |= (uint64_t)(512 >> 4) << 32;                 // stride byte offset between 4-row groups of the reduction
    d |= (uint64_t)1 << 46;                          // descriptor version of this architecture
    d |= (uint64_t)1 << 61;                          // layout: 128-byte swizzle, 32-byte atoms
    return d;
}

// as mma_block32, both operands MN-major: an 8-deep step of the reduction is one 1024-byte group further
template <int BN>
__device__ __forceinline__ void mma_block32_mn(uint32_t tmem, uint32_t a_hi, uint32_t a_lo, uint32_t b_hi, uint32_t b_lo, bool first) {
    constexpr uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
    const uint64_t ah = umma_desc_mn_sw128(a_hi, 4096), al = umma_desc_mn_sw128(a_lo, 4096);
    const uint64_t bh = umma_desc_mn_sw128(b_hi, 4096), bl = umma_desc_mn_sw128(b_lo, 4096);
#pragma unroll
    for (int k = 0; k < T32_BK / 8; ++k) {
        const uint64_t o = (uint64_t)(k * (1024 >> 4));
        umma_tf32(tmem, ah + o, bh + o, idesc, (!first || k > 0) ? 1u : 0u);
        umma_tf32(tmem, ah + o, bl + o, idesc, 1u);
        umma_tf32(tmem, al + o, bh + o, idesc, 1u);
    }
}

// Eight warps write the lo parts (two per scheduler hide each other's shared-memory latency); four of them go on
// to the epilogue.
constexpr int WG32_CONV = 256, WG32_THREADS = 64 + WG32_CONV;

template <int BN>
__global__ void __launch_bounds__(WG32_THREADS) tc32_wgrad_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY,
                                                                const __grid_constant__ CUtensorMap mapD, const T32Params p) {
    using L = Wg32Smem<BN>;
    constexpr uint32_t A_BYTES = L::A_BYTES, B_BYTES = L::B_BYTES, STAGE_BYTES = L::STAGE_BYTES, SLAB = 32 * 32 * 4;
    constexpr int NSTG = L::NSTG;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ __align__(8) unsigned long long bars[3 * NSTG + 1];
    __shared__ uint32_t tmem_base;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * TC_BM, n0 = blockIdx.y * BN, split = blockIdx.z;
    const int kbeg = split * p.rows_per_split, kend = min(p.K, kbeg + p.rows_per_split);
    const int num_kb = (kend - kbeg + T32_BK - 1) / T32_BK;
    // slabs wholly beyond the matrix are neither loaded nor split (they are cleared once in every stage)
    const int slabsA = min(TC_BM / 32, (p.M - m0 + 31) / 32), slabsB = min(BN / 32, (p.N - n0 + 31) / 32);
    const uint32_t tx_bytes = (uint32_t)(slabsA + slabsB) * SLAB;
    const uint32_t full0 = smem_u32(&bars[0]), ready0 = smem_u32(&bars[NSTG]), empty0 = smem_u32(&bars[2 * NSTG]), accum = smem_u32(&bars[3 * NSTG]);

    if (threadIdx.x == 0) {
        tma_prefetch_map(&mapX); tma_prefetch_map(&mapY); tma_prefetch_map(&mapD);
        for (int s = 0; s < NSTG; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(ready0 + 8 * s, WG32_CONV); mbar_init(empty0 + 8 * s, 1); }
        mbar_init(accum, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base)), "r"((uint32_t)BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_base;
    grid_dep_sync();

    if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % NSTG;
                const uint32_t ph = (kb / NSTG) & 1;
                if (kb >= NSTG && !mbar_wait(empty0 + 8 * s, ph ^ 1, p.err, 11)) break;     // the MMAs that read this stage are done
                const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + 2 * A_BYTES;
                const int k = kbeg + kb * T32_BK;
                mbar_expect_tx(full0 + 8 * s, tx_bytes);
                for (int t = 0; t < slabsA; ++t) tma_load_2d(sa + t * SLAB, &mapX, m0 + 32 * t, k, full0 + 8 * s);
                for (int t = 0; t < slabsB; ++t) tma_load_2d(sb + t * SLAB, &mapY, n0 + 32 * t, k, full0 + 8 * s);
                issued = kb + 1;
            }
            if (*((volatile int*)p.err) != 0) {
                for (int kb = max(0, issued - NSTG); kb < issued; ++kb) {
                    const unsigned long long t0 = gtime();
                    while (!mbar_test(full0 + 8 * (kb % NSTG), (kb / NSTG) & 1) && gtime() - t0 < 1000000ull) __nanosleep(128);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            bool ok = true;
            for (int kb = 0; kb < num_kb && ok; ++kb) {
                const int s = kb % NSTG;
                ok = mbar_wait(ready0 + 8 * s, (kb / NSTG) & 1, p.err, 12);            // landed, split and visible
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + 2 * A_BYTES;
                mma_block32_mn<BN>(tmem, sa, sa + A_BYTES, sb, sb + B_BYTES, kb == 0);
                umma_commit(empty0 + 8 * s);
            }
            if (ok) umma_commit(accum);
        }
    } else {
        const int t = threadIdx.x - 64;
        bool ok = true;
        if (slabsA < TC_BM / 32 || slabsB < BN / 32) {
            // clear the slabs that no load will ever fill, hi and lo, in every stage
            const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int s = 0; s < NSTG; ++s) {
                uint8_t* st = smem + s * STAGE_BYTES;
                for (int i = slabsA * SLAB + t * 16; i < (int)A_BYTES; i += WG32_CONV * 16) { *reinterpret_cast<float4*>(st + i) = z; *reinterpret_cast<float4*>(st + A_BYTES + i) = z; }
                for (int i = slabsB * SLAB + t * 16; i < (int)B_BYTES; i += WG32_CONV * 16) { *reinterpret_cast<float4*>(st + 2 * A_BYTES + i) = z; *reinterpret_cast<float4*>(st + 2 * A_BYTES + B_BYTES + i) = z; }
            }
        }
        // a batch norm applied to one operand as it is split: this thread's channels are the same in every block of the reduction
        const int xop = p.xf.scale != nullptr ? p.xf_operand : 0;
        Xf4 xc[4];
        bool xok[4] = {false, false, false, false};
        const int xrow = t >> 3;
        if (xop) {
            const int cw = 8 * (((t & 7) >> 1) ^ (xrow & 3)) + 4 * (t & 1);
            const int o0 = xop == 1 ? m0 : n0, lim = xop == 1 ? p.M : p.N, nsl = xop == 1 ? slabsA : slabsB;
#pragma unroll
            for (int n = 0; n < 4; ++n) {
                const int ch = o0 + 32 * n + cw;
                xok[n] = n < nsl && ch < lim;
                xc[n].load(p.xf, ch, xok[n]);
            }
        }
        for (int kb = 0; kb < num_kb && ok; ++kb) {
            const int s = kb % NSTG;
            ok = mbar_wait(full0 + 8 * s, (kb / NSTG) & 1, p.err, 13);
            if (!ok) break;
            uint8_t* st = smem + s * STAGE_BYTES;
            const bool row_ok = kbeg + kb * T32_BK + xrow < kend;
            if (xop == 1) xform_split_slabs_mn(st, st + A_BYTES, slabsA, t, xc, xok, p.xf.lo, p.xf.hi, row_ok);
            else split_tile(st, st + A_BYTES, slabsA * SLAB, t, WG32_CONV);
            if (xop == 2) xform_split_slabs_mn(st + 2 * A_BYTES, st + 2 * A_BYTES + B_BYTES, slabsB, t, xc, xok, p.xf.lo, p.xf.hi, row_ok);
            else split_tile(st + 2 * A_BYTES, st + 2 * A_BYTES + B_BYTES, slabsB * SLAB, t, WG32_CONV);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // generic-proxy writes -> visible to the tensor cores
            mbar_arrive(ready0 + 8 * s);
        }
        if (warp < 6) {                                                         // warps 2..5 own the four lane quarters of tensor memory
            const bool have = ok && (num_kb > 0 ? mbar_wait(accum, 0, p.err, 14) : true);
            epilogue32<BN>(smem, tmem, &mapD, p, nullptr, m0, n0, split, num_kb, have);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)BN) : "memory");
}

// rows x cols float matrix, cols contiguous; box = 32 columns x box_rows rows, 128-byte swizzle (of 16-byte pieces unless told otherwise), zero fill
bool make_map_f32(CUtensorMap* map, const void* base, long long rows, long long cols, int box_rows, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
    const cuuint32_t box[2] = {(cuuint32_t)T32_BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// output [S][rows][cols] floats; box = 32 columns x 128 rows x 1, 128-byte swizzle (stores clip at the edges)
bool make_map_out(CUtensorMap* map, const void* base, long long S, long long rows, long long cols) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)S};
    const cuuint64_t strides[2] = {(cuuint64_t)cols * 4, (cuuint64_t)rows * cols * 4};
    const cuuint32_t box[3] = {32, (cuuint32_t)TC_BM, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int STAGES>
bool launch32(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& ml, const CUtensorMap& md, const T32Params& p, dim3 grid, cudaStream_t st) {
    constexpr int ring = STAGES * 2 * (TC_BM * T32_BK * 4 + BN * T32_BK * 4);
    constexpr int stage_out = TC_BM * BN * 4;                         // the epilogue reuses the ring as its staging area
    constexpr int smem = (ring > stage_out ? ring : stage_out) + 1024;
    if (cudaFuncSetAttribute(tc32_kernel<BN, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return false;
    launch(tc32_kernel<BN, STAGES>, grid, dim3(TC_THREADS), smem, st, ma, mb, ml, md, p);
    return true;
}

template <int BN>
bool launch32_wgrad(const CUtensorMap& mx, const CUtensorMap& my, const CUtensorMap& md, const T32Params& p, dim3 grid, cudaStream_t st) {
    constexpr int smem = Wg32Smem<BN>::TOTAL;
    static_assert(Wg32Smem<BN>::NSTG >= 2 && Wg32Smem<BN>::NSTG * (int)Wg32Smem<BN>::STAGE_BYTES >= TC_BM * BN * 4, "shared-memory plan");
    if (cudaFuncSetAttribute(tc32_wgrad_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return false;
    launch(tc32_wgrad_kernel<BN>, grid, dim3(WG32_THREADS), smem, st, mx, my, md, p);
    return true;
}

// The tensor core works on 128 x BN tiles whatever part of them is padding, so the weight gradient is computed as
// dW or as dW^T, whichever pads less: the wider of (cin, cout) goes to the 128-row side.  A transposed result is
// put right by the second pass, which then always runs.
struct Wg32Plan { int S, rows_per_split, BN, swap; };
static inline int bn_for(int n) { return n > 64 ? 128 : (n > 32 ? 64 : 32); }
static inline long long mma_area(int m, int n) {
    const int bn = bn_for(n);
    return (long long)((m + TC_BM - 1) / TC_BM) * TC_BM * ((n + bn - 1) / bn) * bn;
}
Wg32Plan plan_wgrad32(long long R, int Mo, int No) {
    Wg32Plan w;
    w.swap = mma_area(No, Mo) < mma_area(Mo, No) ? 1 : 0;
    const int m = w.swap ? No : Mo, n = w.swap ? Mo : No;
    w.BN = bn_for(n);
    const long long tiles = (long long)((m + TC_BM - 1) / TC_BM) * ((n + w.BN - 1) / w.BN);
    // as many blocks as the SMs hold at once (two per SM up to 64-wide tiles, one for 128-wide: see Wg32Smem), no second wave
    const long long per_sm = w.BN <= 64 ? 2 : 1;
    long long S = (per_sm * sm_count()) / tiles;
    const long long maxS = (R + 255) / 256;
    long long cap = (2LL << 20) / ((long long)Mo * No);                     // partial sums cost traffic too: at most 2 Mi floats
    if (cap < 1) cap = 1;
    if (S > maxS) S = maxS;
    if (S > cap) S = cap;
    if (S < 1) S = 1;
    const long long rps = ((R + S - 1) / S + 31) / 32 * 32;
    w.rows_per_split = (int)rps;
    w.S = (int)((R + rps - 1) / rps);
    return w;
}

// out[i][j] = sum_z partial[z][j][i]: the slices are [cols][rows] (the transpose of out[rows][cols]).  One block per
// 32 x 32 tile of out: thread (x, y) reads element (j0 + y + 8 q, i0 + x) of the slices z = y', y' + 4, ... for q = 0..3
// (reads run along the slices' contiguous dimension), the four runs of slices are added in run order, and the tile is
// turned in shared memory so that the stores are contiguous too.  Block (32, 8, 4): z = slice run.
__global__ void __launch_bounds__(1024) slice_sum_transposed_kernel(const float* __restrict__ partial, int S, int rows, int cols, float* __restrict__ out) {
    grid_dep_sync();
    __shared__ float tile[4][32][33];
    const long long count = (long long)rows * cols;
    const int i0 = blockIdx.x * 32, j0 = blockIdx.y * 32;            // out rows i0.., out columns j0..
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    const int i = i0 + threadIdx.x;
    for (int z = threadIdx.z; z < S; z += 4) {
        const float* sl = partial + (long long)z * count;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int j = j0 + threadIdx.y + 8 * q;
            if (j < cols && i < rows) acc[q] += sl[(long long)j * rows + i];
        }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) tile[threadIdx.z][threadIdx.y + 8 * q][threadIdx.x] = acc[q];
    __syncthreads();
    if (threadIdx.z == 0) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int io = i0 + threadIdx.y + 8 * q, jo = j0 + threadIdx.x;
            if (io < rows && jo < cols) {
                const int a = threadIdx.x, b = threadIdx.y + 8 * q;
                out[(long long)io * cols + jo] = (tile[0][a][b] + tile[1][a][b]) + (tile[2][a][b] + tile[3][a][b]);
            }
        }
    }
}

}  // namespace

bool tc32_supported(int M, int N, int K, const void* A, const void* B, const void* D, const void* addend) {
    auto a16 = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; };
    return M >= 1 && N % 4 == 0 && K % 4 == 0 && N >= 4 && K >= 4 && a16(A) && a16(B) && a16(D) && a16(addend) && encode_fn() != nullptr;
}

constexpr int max_stages32(int BN) {
    const int n = (226 * 1024) / (2 * (TC_BM * T32_BK * 4 + BN * T32_BK * 4));
    return n > 4 ? 4 : n;
}

// blocks of tc32_kernel<BN, stages> that an SM holds at once: shared memory (ring or the epilogue's staging tile,
// whichever is larger), tensor-memory columns, threads
static int resident32(int BN, int stages) {
    const int ring = stages * 2 * (TC_BM * T32_BK * 4 + BN * T32_BK * 4), stage_out = TC_BM * BN * 4;
    const int smem = (ring > stage_out ? ring : stage_out) + 1024 + 512;
    int f = (227 * 1024) / smem;
    f = std::min(f, 512 / BN);
    f = std::min(f, 2048 / TC_THREADS);
    return f < 1 ? 1 : f;
}

template <int BN>
bool launch32_stages(int stages, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& ml, const CUtensorMap& md, const T32Params& p, dim3 grid,
                     cudaStream_t st) {
    constexpr int MAXS = max_stages32(BN);
    if (stages > MAXS) stages = MAXS;
    if (stages <= 1) return launch32<BN, 1>(ma, mb, ml, md, p, grid, st);
    if (stages == 2) return launch32<BN, 2>(ma, mb, ml, md, p, grid, st);
    if constexpr (MAXS >= 3) { if (stages == 3) return launch32<BN, 3>(ma, mb, ml, md, p, grid, st); }
    if constexpr (MAXS >= 4) { if (stages == 4) return launch32<BN, 4>(ma, mb, ml, md, p, grid, st); }
    return false;
}

// out = addend + sum over S slices, slice order fixed
__global__ void __launch_bounds__(256) slice_sum_kernel(const float4* __restrict__ part, int S, long long count4, const float4* __restrict__ addend,
                                                        float4* __restrict__ out) {
    grid_dep_sync();
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count4) return;
    float4 a = part[i];
    for (int s = 1; s < S; ++s) { const float4 v = part[(long long)s * count4 + i]; a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w; }
    if (addend) { const float4 v = addend[i]; a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w; }
    out[i] = a;
}

// Tile width, reduction slices and ring depth of a product D[M,N] over K, chosen together by a small cost model.
// What it weighs: (i) blocks beyond what the SMs hold at once run as a second wave, so the number of blocks
// (tiles x slices) is matched to the resident capacity, which the ring depth sets through shared memory; (ii) a
// block's reduction is a serial chain (load, split, multiply) per 32-wide step unless the ring has two stages or
// more; (iii) blocks sharing an SM share its shared-memory bandwidth; (iv) slices cost a second kernel that adds
// them in order.  Times in microseconds, fitted to per-launch times measured on config 2.
struct G32Plan { int BN, S, rps, stages; };
G32Plan plan_gemm32(int M, int N, int K) {
    const int sms = sm_count(), mt = (M + TC_BM - 1) / TC_BM, nkb = (K + T32_BK - 1) / T32_BK;
    // tile width: the widest that does not pad the columns more than a narrower one would (144, 192, 576 or 960 columns
    // leave a 128-wide last tile mostly empty), narrower while the tiles are fewer than the SMs (with eight or more row
    // tiles not below 64 columns: the MMAs of a 32-wide tile read the 128-row operand for a quarter of the output)
    int BN0 = N > 64 ? 128 : (N > 32 ? 64 : 32);
    if (BN0 == 128 && (N + 63) / 64 * 64 < (N + 127) / 128 * 128) BN0 = 64;
    const int narrowest = mt >= 8 ? 64 : 32;
    while (BN0 > narrowest && (long long)mt * ((N + BN0 - 1) / BN0) < sms) BN0 >>= 1;
    G32Plan best{BN0, 1, nkb * T32_BK, 1};
    double best_t = 1e30;
    for (int BN = BN0; BN <= BN0; BN *= 2) {
        const long long tiles = (long long)mt * ((N + BN - 1) / BN);
        const double t0 = 3.0 + BN / 64.0, t_share = 0.3 + 0.1 * BN / 64.0;
        const int maxst = max_stages32(BN);
        for (int S = 1; S <= 8; ++S) {
            const int kbps = (nkb + S - 1) / S, slices = (nkb + kbps - 1) / kbps;
            if (slices != S || (S > 1 && kbps < 2)) continue;
            if (S > 1 && (long long)S * M * N > (4LL << 20)) continue;      // partial sums cost traffic too
            for (int st = 1; st <= maxst && st <= kbps; ++st) {
                const int fit = resident32(BN, st);
                const long long ctas = tiles * S, slots = (long long)sms * fit;
                const long long waves = (ctas + slots - 1) / slots;
                const double conc = (double)std::min<long long>(fit, (ctas + sms - 1) / sms);
                // a block's serial chain per 32-wide step: with a ring of `st` stages that many loads are in flight ahead of the split
                static const double per_step[5] = {0.0, 1.6, 1.0, 0.7, 0.55};
                const double chain = kbps * per_step[st], shared = conc * kbps * t_share;
                double t = waves * (t0 + (chain > shared ? chain : shared));
                if (S > 1) t += 2.5 + (double)(S + 1) * M * N * 4.0 / 3.0e6;
                if (t < best_t - 1e-9) { best_t = t; best = G32Plan{BN, S, kbps * T32_BK, st}; }
            }
        }
    }
    return best;
}

// D[M,N] = A[M,K] * B[N,K]^T (+ addend), float in and out, split-tf32 arithmetic; both operands with K contiguous.
// stats (nullable): the output feeds a batch norm whose fold plan is stats->fold; the partial sums of its statistics go
// to stats->partial, from the epilogue of the product kernel (one entry per 128-row tile) or from the kernel that adds
// the reduction slices, and *stats->out describes them.
bool tc32_gemm(const float* A, const float* B, const float* B_lo, const float* addend, float* D, float* scratch, int M, int N, int K, int* err, cudaStream_t st,
               const ColStatsReq* stats, const BnXform* a_xform) {
    G32Plan g = plan_gemm32(M, N, K);
    if (g.S > 1 && !scratch) { g.S = 1; g.rps = (K + T32_BK - 1) / T32_BK * T32_BK; g.stages = 4; }
    const int BN = g.BN;
    float* out = g.S > 1 ? scratch : D;
    CUtensorMap ma, mb, ml, md;
    if (!make_map_f32(&ma, A, M, K, TC_BM) || !make_map_out(&md, out, g.S, M, N) || !make_map_f32(&mb, B, N, K, BN)) return false;
    if (B_lo) { if (!make_map_f32(&ml, B_lo, N, K, BN)) return false; }
    else ml = mb;
    T32Params p{out, g.S > 1 ? nullptr : addend, M, N, K, g.rps, B_lo ? 1 : 0, err, (stats && g.S == 1) ? stats->partial : nullptr,
                a_xform ? *a_xform : BnXform{nullptr, nullptr, nullptr, 0.f, 0.f}, a_xform ? 1 : 0};
    const dim3 grid((N + BN - 1) / BN, (M + TC_BM - 1) / TC_BM, g.S);
    const int nkb = g.rps / T32_BK, stages = g.stages > nkb ? (nkb < 1 ? 1 : nkb) : g.stages;
    bool ok;
    if (BN == 128) ok = launch32_stages<128>(stages, ma, mb, ml, md, p, grid, st);
    else if (BN == 64) ok = launch32_stages<64>(stages, ma, mb, ml, md, p, grid, st);
    else ok = launch32_stages<32>(stages, ma, mb, ml, md, p, grid, st);
    if (ok && stats) *stats->out = PartialSums{stats->partial, (int)grid.y, 1};
    if (ok && g.S > 1 && stats && !addend && slice_sum_stats(scratch, g.S, D, M, N, *stats->fold, stats->partial, stats->out, st)) return true;
    if (ok && g.S > 1) {
        if (stats) stats->out->entries = 0;          // none were produced
        const long long count4 = (long long)M * N / 4;
        launch(slice_sum_kernel, dim3((unsigned)((count4 + 255) / 256)), dim3(256), 0, st, reinterpret_cast<const float4*>(scratch), g.S, count4,
               reinterpret_cast<const float4*>(addend), reinterpret_cast<float4*>(D));
    }
    return ok;
}

size_t tc32_gemm_scratch_floats(int M, int N, int K) {
    const G32Plan g = plan_gemm32(M, N, K);
    return g.S > 1 ? (size_t)g.S * M * N : 0;
}

size_t tc32_wgrad_scratch_floats(long long R, int Mo, int No) {
    const Wg32Plan w = plan_wgrad32(R, Mo, No);
    return (w.S > 1 || w.swap) ? (size_t)w.S * Mo * No : 0;
}

// dW[Mo][No] = X[R][Mo]^T * dY[R][No], second pass included; false: nothing launched
bool tc32_wgrad(const float* X, const float* dY, float* dW, float* scratch, long long R, int Mo, int No, int* err, cudaStream_t st, const BnXform* x_xform) {
    const Wg32Plan w = plan_wgrad32(R, Mo, No);
    const bool two_pass = w.S > 1 || w.swap;
    if (two_pass && !scratch) return false;
    const float* A = w.swap ? dY : X;
    const float* B = w.swap ? X : dY;
    const int m = w.swap ? No : Mo, n = w.swap ? Mo : No;
    CUtensorMap mx, my, md;
    float* out = two_pass ? scratch : dW;
    if (!make_map_f32(&mx, A, R, m, 32, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B) || !make_map_f32(&my, B, R, n, 32, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B) || !make_map_out(&md, out, w.S, m, n)) return false;
    T32Params p{out, nullptr, m, n, (int)R, w.rows_per_split, 0, err, nullptr,
                x_xform ? *x_xform : BnXform{nullptr, nullptr, nullptr, 0.f, 0.f}, x_xform ? (w.swap ? 2 : 1) : 0};
    const dim3 grid((m + TC_BM - 1) / TC_BM, (n + w.BN - 1) / w.BN, w.S);
    bool ok;
    if (w.BN == 128) ok = launch32_wgrad<128>(mx, my, md, p, grid, st);
    else if (w.BN == 64) ok = launch32_wgrad<64>(mx, my, md, p, grid, st);
    else ok = launch32_wgrad<32>(mx, my, md, p, grid, st);
    if (!ok) return false;
    const long long count = (long long)Mo * No;
    if (w.swap) launch(slice_sum_transposed_kernel, dim3((Mo + 31) / 32, (No + 31) / 32), dim3(32, 8, 4), 0, st, (const float*)scratch, w.S, Mo, No, dW);
    else if (w.S > 1) split_reduce_f32(scratch, w.S, count, dW, st);
    return true;
}

}  // namespace ftp
