// bf16 contractions on the 5th-generation tensor cores (sm_100a): D[M,N] = A[M,K] * B[N,K]^T with both
// operands K-major in global memory, float accumulation in tensor memory, bf16 output.
//
// One CTA computes one 128 x BN output tile.  Warp 0 (one elected thread) streams 128 x 64 and BN x 64
// operand tiles into a ring of shared-memory stages with TMA (128-byte swizzle, out-of-range rows and
// columns filled with zeros, no multicast); warp 1 allocates BN columns of tensor memory and, through one
// thread, issues tcgen05.mma (M = 128, N = BN, K = 16) four times per stage, releasing the stage with
// tcgen05.commit; warps 2-5 wait for the last commit, read the accumulator with tcgen05.ld (each warp its
// own 32 lanes), add the optional addend, convert and store.  Every wait on an mbarrier is bounded: when it
// runs out the kernel records a code in an error word, lets its own copies land, frees its tensor memory
// and returns; the host reports FTP_ETIMEOUT.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include "gemm_tc_common.cuh"

namespace ftp {
namespace tc {
EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

}  // namespace tc
using namespace tc;
namespace {

struct TcParams {
    __nv_bfloat16* D;
    const __nv_bfloat16* addend;   // nullable, shaped like D
    int M, N, K;                   // K: reduction length (conv: 9 * channels)
    int* err;
    ConvTap conv;
    float* partial;                // reduction cut into gridDim.z slices: partial sums [slice][M][N] (float) instead of D
    int kb_per_slice;              // 64-wide reduction blocks per slice
};

// NSTG: depth of the operand ring.  A block's reduction advances one stage per (load latency / NSTG), so products with
// one block per SM or fewer take a ring as deep as shared memory holds, products with several blocks per SM a short one.
template <int BN, int NSTG>
__global__ void __launch_bounds__(TC_THREADS) tc_gemm_tn_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                                                                const __grid_constant__ CUtensorMap mapD, const TcParams p) {
    constexpr int TC_STAGES = NSTG;
    constexpr uint32_t A_BYTES = TC_BM * TC_BK * 2, B_BYTES = BN * TC_BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ __align__(8) unsigned long long bars[2 * TC_STAGES + 1];
    __shared__ uint32_t tmem_base;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * BN, m0 = blockIdx.y * TC_BM;
    const int all_kb = (p.K + TC_BK - 1) / TC_BK;
    const bool sliced = p.partial != nullptr;
    const int kb0 = sliced ? blockIdx.z * p.kb_per_slice : 0;
    const int num_kb = sliced ? max(0, min(all_kb, kb0 + p.kb_per_slice) - kb0) : all_kb;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[TC_STAGES]), accum = smem_u32(&bars[2 * TC_STAGES]);

    if (threadIdx.x == 0) {
        tma_prefetch_map(&mapA); tma_prefetch_map(&mapB);
        if (BN >= 64) tma_prefetch_map(&mapD);
        for (int s = 0; s < TC_STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
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
            // ---- producer: TMA loads into the stage ring ----
            int issued = 0;
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % TC_STAGES;
                const uint32_t ph = (kb / TC_STAGES) & 1;
                if (kb >= TC_STAGES && !mbar_wait(empty0 + 8 * s, ph ^ 1, p.err, 1)) break;
                const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + A_BYTES;
                const int gkb = kb0 + kb;                    // block of the whole reduction
                mbar_expect_tx(full0 + 8 * s, STAGE_BYTES);
                if (!p.conv.enabled) {
                    tma_load_2d(sa, &mapA, gkb * TC_BK, m0, full0 + 8 * s);
                    tma_load_2d(sb, &mapB, gkb * TC_BK, n0, full0 + 8 * s);
                } else {
                    const int tap = gkb / p.conv.chunks, cc = gkb - tap * p.conv.chunks, r = tap / 3, sx = tap - 3 * r;
                    const int hw = p.conv.H * p.conv.W, img = m0 / hw, h0 = (m0 - img * hw) / p.conv.W;
                    const int dh = p.conv.flip ? 1 - r : r - 1, dw = p.conv.flip ? 1 - sx : sx - 1;
                    tma_load_4d(sa, &mapA, cc * 64, dw, h0 + dh, img, full0 + 8 * s);
                    tma_load_2d(sb, &mapB, cc * 64, tap * p.conv.b_rows + n0, full0 + 8 * s);
                }
                issued = kb + 1;
            }
            if (*((volatile int*)p.err) != 0) {
                // error path: let the copies already issued land before the block's memory is released
                for (int kb = max(0, issued - TC_STAGES); kb < issued; ++kb) {
                    const unsigned long long t0 = gtime();
                    while (!mbar_test(full0 + 8 * (kb % TC_STAGES), (kb / TC_STAGES) & 1) && gtime() - t0 < 1000000ull) __nanosleep(128);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issuer ----
            constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
            bool ok = true;
            for (int kb = 0; kb < num_kb && ok; ++kb) {
                const int s = kb % TC_STAGES;
                const uint32_t ph = (kb / TC_STAGES) & 1;
                ok = mbar_wait(full0 + 8 * s, ph, p.err, 2);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + A_BYTES;
                const uint64_t ad = umma_desc_k_sw128(sa), bd = umma_desc_k_sw128(sb);
#pragma unroll
                for (int k = 0; k < TC_BK / 16; ++k)                 // 16 bf16 = 32 bytes along K inside the swizzle atom
                    umma_bf16(tmem, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 2), idesc, (kb > 0 || k > 0) ? 1u : 0u);
                umma_commit(empty0 + 8 * s);                         // frees the stage once these MMAs have read it
            }
            if (ok) umma_commit(accum);                              // accumulator complete
        }
    } else {
        // ---- epilogue: warps 2..5 own tensor-memory lanes 32*(warp%4) .. +31 ----
        const int q = warp & 3;
        const bool have = num_kb > 0 ? mbar_wait(accum, 0, p.err, 3) : true;         // every stage has been consumed by now: the ring is free
        if (have) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int m = m0 + q * 32 + lane;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t r[32];
                if (num_kb > 0) tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32), r);
                else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) r[e] = 0u;
                }
                const int nb = n0 + c * 32;
                if (sliced) {                                        // float partial sums of this slice, added up by a second kernel
                    if (m < p.M) {
                        float* prow = p.partial + ((long long)blockIdx.z * p.M + m) * p.N + nb;
#pragma unroll
                        for (int g = 0; g < 8; ++g)
                            if (nb + g * 4 < p.N)
                                *reinterpret_cast<float4*>(prow + g * 4) = make_float4(__uint_as_float(r[g * 4]), __uint_as_float(r[g * 4 + 1]),
                                                                                      __uint_as_float(r[g * 4 + 2]), __uint_as_float(r[g * 4 + 3]));
                    }
                    continue;
                }
                if (m < p.M) {
                    __nv_bfloat16* drow = p.D + (long long)m * p.N + nb;
                    const __nv_bfloat16* arow = p.addend ? p.addend + (long long)m * p.N + nb : nullptr;
#pragma unroll
                    for (int g = 0; g < 4; ++g) {                    // 8 columns = 16 bytes per store
                        if (nb + g * 8 < p.N) {
                            float v[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(r[g * 8 + e]);
                            if (arow) {
                                const uint4 a = __ldg(reinterpret_cast<const uint4*>(arow + g * 8));
                                const unsigned au[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) { v[2 * e] += __uint_as_float(au[e] << 16); v[2 * e + 1] += __uint_as_float(au[e] & 0xffff0000u); }
                            }
                            unsigned o[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) { const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]); o[e] = *reinterpret_cast<const unsigned*>(&h); }
                            if (BN >= 64) {
                                // staged for one TMA store per 128 x 64 piece: 128-byte rows, 16-byte chunk index XOR row % 8
                                const int row = q * 32 + lane, j = (c & 1) * 4 + g;
                                *reinterpret_cast<uint4*>(smem + (c >> 1) * (TC_BM * 128) + row * 128 + ((j ^ (row & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                            } else
                                *reinterpret_cast<uint4*>(drow + g * 8) = make_uint4(o[0], o[1], o[2], o[3]);
                        }
                    }
                }
            }
            if (BN >= 64 && !sliced) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        if (BN >= 64) {
            // whole 128-byte lines leave through TMA (clipped at the edges of D) instead of 16-byte pieces per thread
            asm volatile("bar.sync 1, 128;" ::: "memory");                  // the four epilogue warps
            if (have && !sliced && threadIdx.x == 64) {
#pragma unroll 1
                for (int c = 0; c < BN / 64; ++c)
                    if (n0 + c * 64 < p.N)
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                                     ::"l"(&mapD), "r"(n0 + c * 64), "r"(m0), "r"(smem_u32(smem + c * (TC_BM * 128))) : "memory");
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // shared memory may be released after this
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)BN) : "memory");
}

// ---- persistent variant ------------------------------------------------------------------------------------------
// One block per SM walks the output tiles t = blockIdx.x, + gridDim.x, ...  The operand ring never drains between
// tiles; the accumulator rotates through TCP_TEAMS BN-column parts of the block's tensor memory, and as many teams of
// four epilogue warps take the tiles in turn (team g reads part g), so the read-out, conversion and store of a tile
// overlap the loads and MMAs of the tiles after it.  What a tile costs is then the slower of its loads and a
// TCP_TEAMS-th of an epilogue, not their sum plus the block's set-up -- which is what bounded the products with a short
// reduction and many tiles (the 1x1 convolutions on large maps; timestamps inside the kernel: 0.4 us from the first MMA
// to the commit, about 1 us until the team has seen it, 1 us to read and convert 128 x 128, 0.4 us to hand the tile to
// TMA -- with two teams 1.2 us per tile).  Barriers: full / empty per stage as above; accf[g] (the MMAs of a tile for part
// g have completed), acce[g] (the four warps of team g have read part g).  No reduction slices here.
constexpr int TCP_TEAMS = 4;
constexpr int TCP_THREADS = 64 + 128 * TCP_TEAMS;
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]),
          "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
          "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_one(uint32_t bar) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory"); }

template <int BN, int NSTG>
__global__ void __launch_bounds__(TCP_THREADS, 1) tc_gemm_tn_persistent_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                                                                               const __grid_constant__ CUtensorMap mapD, const TcParams p, int tiles_n,
                                                                               long long total_tiles) {
    constexpr uint32_t A_BYTES = TC_BM * TC_BK * 2, B_BYTES = BN * TC_BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
    constexpr uint32_t OUT_BYTES = BN >= 64 ? TC_BM * BN * 2 : 0;        // a team's staging tile for the TMA store
    constexpr uint32_t TMEM_COLS = TCP_TEAMS * BN;
    static_assert(TMEM_COLS >= 32 && TMEM_COLS <= 512 && (TMEM_COLS & (TMEM_COLS - 1)) == 0, "tensor-memory allocation is a power of two");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* stage_out = smem + NSTG * STAGE_BYTES;
    __shared__ __align__(8) unsigned long long bars[2 * NSTG + 2 * TCP_TEAMS];
    __shared__ uint32_t tmem_base;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (p.K + TC_BK - 1) / TC_BK;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[NSTG]), accf0 = smem_u32(&bars[2 * NSTG]), acce0 = smem_u32(&bars[2 * NSTG + TCP_TEAMS]);

    if (threadIdx.x == 0) {
        tma_prefetch_map(&mapA); tma_prefetch_map(&mapB);
        if (BN >= 64) tma_prefetch_map(&mapD);
        for (int s = 0; s < NSTG; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int g = 0; g < TCP_TEAMS; ++g) { mbar_init(accf0 + 8 * g, 1); mbar_init(acce0 + 8 * g, 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_base;
    grid_dep_sync();

    if (warp == 0) {
        if (lane == 0) {
            // ---- producer ----
            long long it = 0;                                        // stages filled so far, over all tiles
            bool ok = true;
            for (long long t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const int m0 = (int)(t / tiles_n) * TC_BM, n0 = (int)(t % tiles_n) * BN;
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = (int)(it % NSTG);
                    const uint32_t ph = (uint32_t)(it / NSTG) & 1u;
                    if (it >= NSTG && !mbar_wait(empty0 + 8 * s, ph ^ 1, p.err, 1)) { ok = false; break; }
                    const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + A_BYTES;
                    mbar_expect_tx(full0 + 8 * s, STAGE_BYTES);
                    if (!p.conv.enabled) {
                        tma_load_2d(sa, &mapA, kb * TC_BK, m0, full0 + 8 * s);
                        tma_load_2d(sb, &mapB, kb * TC_BK, n0, full0 + 8 * s);
                    } else {
                        const int tap = kb / p.conv.chunks, cc = kb - tap * p.conv.chunks, r = tap / 3, sx = tap - 3 * r;
                        const int hw = p.conv.H * p.conv.W, img = m0 / hw, h0 = (m0 - img * hw) / p.conv.W;
                        const int dh = p.conv.flip ? 1 - r : r - 1, dw = p.conv.flip ? 1 - sx : sx - 1;
                        tma_load_4d(sa, &mapA, cc * 64, dw, h0 + dh, img, full0 + 8 * s);
                        tma_load_2d(sb, &mapB, cc * 64, tap * p.conv.b_rows + n0, full0 + 8 * s);
                    }
                }
            }
            if (*((volatile int*)p.err) != 0) {
                // error path: let the copies already issued land before the block's memory is released
                for (long long k = it > NSTG ? it - NSTG : 0; k < it; ++k) {
                    const unsigned long long t0 = gtime();
                    while (!mbar_test(full0 + 8 * (int)(k % NSTG), (uint32_t)(k / NSTG) & 1u) && gtime() - t0 < 1000000ull) __nanosleep(128);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issuer ----
            constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
            long long it = 0;
            bool ok = true;
            int i = 0;                                               // tiles of this block so far
            for (long long t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++i) {
                const int g = i % TCP_TEAMS, j = i / TCP_TEAMS;      // part of the tensor memory, and how often it has been used
                if (j > 0 && !mbar_wait(acce0 + 8 * g, (uint32_t)(j - 1) & 1u, p.err, 4)) { ok = false; break; }   // team g has read the tile before
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = (int)(it % NSTG);
                    const uint32_t ph = (uint32_t)(it / NSTG) & 1u;
                    if (!mbar_wait(full0 + 8 * s, ph, p.err, 2)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + A_BYTES;
                    const uint64_t ad = umma_desc_k_sw128(sa), bd = umma_desc_k_sw128(sb);
                    // 16-wide steps that hold part of the reduction (TMA filled the rest of the block with zeros)
                    const int ksteps = p.conv.enabled ? TC_BK / 16 : min(TC_BK / 16, (p.K - kb * TC_BK + 15) / 16);
#pragma unroll
                    for (int k = 0; k < TC_BK / 16; ++k)
                        if (k < ksteps) umma_bf16(tmem + (uint32_t)(g * BN), ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 2), idesc, (kb > 0 || k > 0) ? 1u : 0u);
                    umma_commit(empty0 + 8 * s);
                }
                if (ok) umma_commit(accf0 + 8 * g);
            }
        }
    } else {
        // ---- epilogue: team g = warps 2 + 4 g .. 5 + 4 g takes the tiles i = g, g + TCP_TEAMS, ...; a warp reads the 32 lanes of its quarter ----
        const int g = (warp - 2) >> 2, q = warp & 3;
        const bool elected = ((warp - 2) & 3) == 0 && lane == 0;     // issues the team's TMA stores
        uint8_t* so = stage_out + g * OUT_BYTES;
        bool ok = true;
        int j = 0;
        for (long long t = blockIdx.x + (long long)g * gridDim.x; t < total_tiles; t += (long long)TCP_TEAMS * gridDim.x, ++j) {
            const int m0 = (int)(t / tiles_n) * TC_BM, n0 = (int)(t % tiles_n) * BN;
            // whether the tile arrived is decided per warp (the tensor-memory loads below are warp-wide) and, where the team
            // meets at a barrier anyway, per team: nobody is left waiting at a barrier that the others gave up on
            ok = __all_sync(0xffffffffu, mbar_wait(accf0 + 8 * g, (uint32_t)j & 1u, p.err, 3));
            if (BN >= 64) {
                // the staging tile is free once the store of the team's tile before has read it
                if (elected) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                uint32_t all_ok;
                asm volatile("{\n.reg .pred p, q;\nsetp.ne.b32 p, %1, 0;\nbar.red.and.pred q, %2, 128, p;\nselp.b32 %0, 1, 0, q;\n}"
                             : "=r"(all_ok) : "r"((uint32_t)ok), "r"(1 + g) : "memory");
                ok = all_ok != 0;
            }
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int m = m0 + q * 32 + lane;
            constexpr int CPR = BN >= 64 ? 2 : 1;                    // 32-column chunks read per round trip to the tensor memory
#pragma unroll 1
            for (int c0 = 0; c0 < BN / 32; c0 += CPR) {
                uint32_t rr[CPR][32];
#pragma unroll
                for (int u = 0; u < CPR; ++u) tmem_ld32_issue(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(g * BN + (c0 + u) * 32), rr[u]);
                tmem_ld_wait();
                if (c0 + CPR >= BN / 32) {                           // the part is in registers: the MMAs of a later tile may overwrite it
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    if (lane == 0) mbar_arrive_one(acce0 + 8 * g);
                }
#pragma unroll
                for (int u = 0; u < CPR; ++u) {
                    const int c = c0 + u, nb = n0 + c * 32;
                    if (BN >= 64 || m < p.M) {
                        __nv_bfloat16* drow = p.D + (long long)m * p.N + nb;
                        const __nv_bfloat16* arow = (p.addend && m < p.M) ? p.addend + (long long)m * p.N + nb : nullptr;
#pragma unroll
                        for (int k = 0; k < 4; ++k) {                // 8 columns = 16 bytes per store
                            if (nb + k * 8 < p.N) {
                                float v[8];
#pragma unroll
                                for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(rr[u][k * 8 + e]);
                                if (arow) {
                                    const uint4 a = __ldg(reinterpret_cast<const uint4*>(arow + k * 8));
                                    const unsigned au[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
                                    for (int e = 0; e < 4; ++e) { v[2 * e] += __uint_as_float(au[e] << 16); v[2 * e + 1] += __uint_as_float(au[e] & 0xffff0000u); }
                                }
                                unsigned o[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) { const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]); o[e] = *reinterpret_cast<const unsigned*>(&h); }
                                if (BN >= 64) {
                                    const int row = q * 32 + lane, jj = (c & 1) * 4 + k;
                                    *reinterpret_cast<uint4*>(so + (c >> 1) * (TC_BM * 128) + row * 128 + ((jj ^ (row & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                                } else
                                    *reinterpret_cast<uint4*>(drow + k * 8) = make_uint4(o[0], o[1], o[2], o[3]);
                            }
                        }
                    }
                }
            }
            if (BN >= 64) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                asm volatile("bar.sync %0, 128;" ::"r"(1 + g) : "memory");
                if (elected) {
#pragma unroll 1
                    for (int c = 0; c < BN / 64; ++c)
                        if (n0 + c * 64 < p.N)
                            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                                         ::"l"(&mapD), "r"(n0 + c * 64), "r"(m0), "r"(smem_u32(so + c * (TC_BM * 128))) : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
        }
        if (BN >= 64 && elected) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");      // shared memory may be released after this
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
}

// Shared-memory operand descriptor, MN-major, 128-byte swizzle: a 64 x 64 slab is 64 rows (K) of 128 bytes (64 MN
// elements); 8-row groups are 1024 bytes apart (stride offset), the next 64 MN elements start slab_bytes further
// (leading offset).
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t saddr, uint32_t slab_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFF);
    d |= (uint64_t)((slab_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

struct TcWgParams {
    float* out;          // partials [S][taps][Mo][No] (or the result itself when S == 1)
    int Mo, No;          // output rows (input channels) and columns (output channels)
    int R;               // reduction length: rows of X and dY
    int rows_per_split;  // multiple of 64
    int* err;
    ConvTap conv;        // enabled: grid.z = splits * 9, X is read through a 4-D map shifted by the tap
    int pair;            // conv with Mo <= 64: a block takes two taps, one per 64-row half of its tile (grid.z = splits * 5)
};

// out[z][i][j] = sum over rows r of split z of X[r][i] * dY[r][j].  Both operands are read as they lie in memory
// (channels contiguous), i.e. MN-major; a stage holds 64 reduction rows.
template <int BN>
__global__ void __launch_bounds__(TC_THREADS) tc_wgrad_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY,
                                                              const TcWgParams p) {
    constexpr uint32_t SLAB = 64 * 64 * 2, A_BYTES = 2 * SLAB, B_BYTES = (BN / 64) * SLAB, STAGE_BYTES = A_BYTES + B_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ __align__(8) unsigned long long bars[2 * TC_STAGES + 1];
    __shared__ uint32_t tmem_base;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i0 = blockIdx.x * TC_BM, j0 = blockIdx.y * BN;
    // 64 input channels fill half of the 128-row tile: the other half then takes the next tap (rows 64.. = tap + 1)
    const int taps = p.conv.enabled ? 9 : 1, groups = p.pair ? 5 : taps;
    const int split = blockIdx.z / groups, grp = blockIdx.z - split * groups, tap = p.pair ? 2 * grp : grp;
    const bool second = p.pair && tap + 1 < 9;
    const int rbeg = split * p.rows_per_split, rend = min(p.R, rbeg + p.rows_per_split);
    const int num_kb = (rend - rbeg + 63) / 64;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[TC_STAGES]), accum = smem_u32(&bars[2 * TC_STAGES]);

    if (threadIdx.x == 0) {
        tma_prefetch_map(&mapX); tma_prefetch_map(&mapY);
        for (int s = 0; s < TC_STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
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
                const int s = kb % TC_STAGES;
                const uint32_t ph = (kb / TC_STAGES) & 1;
                if (kb >= TC_STAGES && !mbar_wait(empty0 + 8 * s, ph ^ 1, p.err, 4)) break;
                const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + A_BYTES;
                const int r = rbeg + kb * 64;
                mbar_expect_tx(full0 + 8 * s, (p.pair && !second) ? STAGE_BYTES - SLAB : STAGE_BYTES);
                if (!p.conv.enabled) {
                    tma_load_2d(sa, &mapX, i0, r, full0 + 8 * s);
                    tma_load_2d(sa + SLAB, &mapX, i0 + 64, r, full0 + 8 * s);
                } else {
                    const int tr = tap / 3, ts = tap - 3 * tr;
                    const int hw = p.conv.H * p.conv.W, img = r / hw, h0 = (r - img * hw) / p.conv.W;
                    tma_load_4d(sa, &mapX, i0, ts - 1, h0 + tr - 1, img, full0 + 8 * s);
                    if (!p.pair) tma_load_4d(sa + SLAB, &mapX, i0 + 64, ts - 1, h0 + tr - 1, img, full0 + 8 * s);
                    else if (second) {
                        const int tr2 = (tap + 1) / 3, ts2 = tap + 1 - 3 * tr2;
                        tma_load_4d(sa + SLAB, &mapX, i0, ts2 - 1, h0 + tr2 - 1, img, full0 + 8 * s);
                    }                                                // no second tap: rows 64.. of the tile are never stored
                }
#pragma unroll
                for (int t = 0; t < BN / 64; ++t) tma_load_2d(sb + t * SLAB, &mapY, j0 + 64 * t, r, full0 + 8 * s);
                issued = kb + 1;
            }
            if (*((volatile int*)p.err) != 0) {
                for (int kb = max(0, issued - TC_STAGES); kb < issued; ++kb) {
                    const unsigned long long t0 = gtime();
                    while (!mbar_test(full0 + 8 * (kb % TC_STAGES), (kb / TC_STAGES) & 1) && gtime() - t0 < 1000000ull) __nanosleep(128);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // both operands MN-major: bits 15 and 16
            constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
            bool ok = true;
            for (int kb = 0; kb < num_kb && ok; ++kb) {
                const int s = kb % TC_STAGES;
                const uint32_t ph = (kb / TC_STAGES) & 1;
                ok = mbar_wait(full0 + 8 * s, ph, p.err, 5);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + A_BYTES;
                const uint64_t ad = umma_desc_mn_sw128(sa, SLAB), bd = umma_desc_mn_sw128(sb, SLAB);
#pragma unroll
                for (int k = 0; k < 4; ++k)                           // 16 reduction rows = 2048 bytes further
                    umma_bf16(tmem, ad + (uint64_t)(k * 128), bd + (uint64_t)(k * 128), idesc, (kb > 0 || k > 0) ? 1u : 0u);
                umma_commit(empty0 + 8 * s);
            }
            if (ok) umma_commit(accum);
        }
    } else {
        const int q = warp & 3;
        if (num_kb > 0 ? mbar_wait(accum, 0, p.err, 6) : true) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int row = q * 32 + lane;
            const int i = p.pair ? (row & 63) : i0 + row, otap = p.pair ? tap + (row >> 6) : tap;
            const bool row_ok = i < p.Mo && otap < taps;
            float* orow = p.out + (((long long)split * taps + otap) * p.Mo + i) * p.No;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t r[32];
                if (num_kb > 0) tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32), r);
                else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) r[e] = 0u;
                }
                const int jb = j0 + c * 32;
                if (row_ok) {
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        if (jb + g * 4 < p.No)
                            *reinterpret_cast<float4*>(orow + jb + g * 4) = make_float4(__uint_as_float(r[g * 4]), __uint_as_float(r[g * 4 + 1]),
                                                                                      __uint_as_float(r[g * 4 + 2]), __uint_as_float(r[g * 4 + 3]));
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)BN) : "memory");
}

struct TcWgPlan { int S, rows_per_split; };
// FTP_TC_WG_PAIR=0: one tap per block whatever the channel count (A/B measurements)
static bool wgrad3x3_pairs_taps(int Mo) {
    static int on = -1;
    if (on < 0) { const char* e = std::getenv("FTP_TC_WG_PAIR"); on = (e && std::strcmp(e, "0") == 0) ? 0 : 1; }
    return on != 0 && Mo <= 64;
}
TcWgPlan plan_tc_wgrad(long long R, int Mo, int No) {
    const long long tiles = ((Mo + TC_BM - 1) / TC_BM) * ((No + 127) / 128);
    long long S = (2LL * sm_count() + tiles - 1) / tiles;
    const long long maxS = (R + 511) / 512;                                 // at least 512 rows per split
    long long cap = (8LL << 20) / ((long long)Mo * No);                     // partials within 8 Mi floats
    if (cap < 1) cap = 1;
    if (S > maxS) S = maxS;
    if (S > cap) S = cap;
    if (S < 1) S = 1;
    long long rps = ((R + S - 1) / S + 63) / 64 * 64;
    TcWgPlan w;
    w.rows_per_split = (int)rps;
    w.S = (int)((R + rps - 1) / rps);
    return w;
}

// rows x cols bf16 matrix, cols contiguous; box = 64 columns x box_rows rows, 128-byte swizzle, zero fill
bool make_map_2d(CUtensorMap* map, const void* base, long long rows, long long cols, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// (N, H, W, C) bf16 activation; box = 64 channels x the full width x bh rows x bn images (pix = W*bh*bn pixels)
bool make_map_4d(CUtensorMap* map, const void* base, int N, int H, int W, int C, int pix) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    int bh = pix / W;
    if (bh > H) bh = H;
    const int bn = pix / (W * bh);
    const cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
    const cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)W, (cuuint32_t)bh, (cuuint32_t)bn};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// an image tiles into boxes of `pix` pixels made of whole rows (and whole images when the image is smaller)
bool conv_tiles_ok(int H, int W, int pix) {
    if (W < 1 || W > pix || pix % W != 0) return false;
    const int bh = pix / W;
    if (bh <= H) return H % bh == 0;
    return bh % H == 0;            // several whole images per box
}

// Ring depth and reduction slices of a forward / data-gradient product with `tiles` output tiles and `nkb` 64-wide blocks
// of the reduction.  At most one block per SM: the deepest ring (the reduction then advances at load latency / 6 per
// block instead of / 3).  Far fewer blocks than SMs and a long reduction: cut it into slices (float partial sums,
// added in order by a second kernel).
struct TnPlan { int stages, S, kbps; };
static TnPlan plan_tn(long long tiles, int nkb, long long out_elems) {
    const int sms = sm_count();
    TnPlan pl{tiles <= sms ? 6 : 3, 1, nkb};
    if (tiles * 2 <= sms && nkb >= 16) {
        long long S = sms / tiles;
        if (S > nkb / 8) S = nkb / 8;
        if (S > 8) S = 8;
        const long long cap = (8LL << 20) / std::max<long long>(out_elems, 1);
        if (S > cap) S = cap;
        if (S > 1) {
            pl.kbps = (int)((nkb + S - 1) / S);
            pl.S = (nkb + pl.kbps - 1) / pl.kbps;
        }
    }
    return pl;
}

// 128 x 256 tiles load a third less per multiply-add than 128 x 128 tiles (the products of the wide layers are bound
// by the path from L2 to shared memory, not by the tensor pipe); taken when the output is at least 256 columns wide and
// the wide tiles (times their reduction slices) still occupy most SMs.  FTP_TC_BN256=0 switches them off (A/B).
static bool use_bn256(int M, int N, int K) {
    static int on = -1;
    if (on < 0) { const char* e = std::getenv("FTP_TC_BN256"); on = (e && std::strcmp(e, "0") == 0) ? 0 : 1; }
    if (!on || N < 256) return false;
    const long long tiles = (long long)((N + 255) / 256) * ((M + TC_BM - 1) / TC_BM);
    const TnPlan pl = plan_tn(tiles, (K + TC_BK - 1) / TC_BK, (long long)M * N);
    return tiles * pl.S >= sm_count() / 2;
}

// D = bf16(addend + sum over S float slices), slice order fixed
__global__ void __launch_bounds__(256) slice_sum_bf16_kernel(const float4* __restrict__ part, int S, long long count4, const __nv_bfloat16* __restrict__ addend,
                                                             __nv_bfloat16* __restrict__ out) {
    grid_dep_sync();
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count4) return;
    float4 a = part[i];
    for (int s = 1; s < S; ++s) { const float4 v = part[(long long)s * count4 + i]; a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w; }
    if (addend) {
        const uint2 q = *reinterpret_cast<const uint2*>(addend + i * 4);
        a.x += __uint_as_float(q.x << 16); a.y += __uint_as_float(q.x & 0xffff0000u);
        a.z += __uint_as_float(q.y << 16); a.w += __uint_as_float(q.y & 0xffff0000u);
    }
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(a.z, a.w);
    *reinterpret_cast<uint2*>(out + i * 4) = make_uint2(*reinterpret_cast<const unsigned*>(&lo), *reinterpret_cast<const unsigned*>(&hi));
}

template <int BN, int NSTG>
bool launch_tn_kernel(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& md, const TcParams& p, dim3 grid, cudaStream_t st) {
    constexpr int smem = NSTG * (TC_BM * TC_BK * 2 + BN * TC_BK * 2) + 1024;
    static_assert(NSTG * (TC_BM * TC_BK * 2 + BN * TC_BK * 2) >= TC_BM * BN * 2, "the epilogue stages its tile in the ring");
    if (cudaFuncSetAttribute(tc_gemm_tn_kernel<BN, NSTG>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return false;
    launch(tc_gemm_tn_kernel<BN, NSTG>, grid, dim3(TC_THREADS), smem, st, ma, mb, md, p);
    return true;
}

template <int BN, int NSTG>
bool launch_tn_persistent(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& md, const TcParams& p, cudaStream_t st) {
    constexpr int smem = NSTG * (TC_BM * TC_BK * 2 + BN * TC_BK * 2) + (BN >= 64 ? TCP_TEAMS * TC_BM * BN * 2 : 0) + 1024;
    static_assert(smem + 256 <= 227 * 1024, "ring and staging tiles exceed the shared memory of an SM");
    if (cudaFuncSetAttribute(tc_gemm_tn_persistent_kernel<BN, NSTG>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return false;
    const int tiles_n = (p.N + BN - 1) / BN;
    const long long total = (long long)tiles_n * ((p.M + TC_BM - 1) / TC_BM);
    const unsigned blocks = (unsigned)std::min<long long>(total, sm_count());
    launch(tc_gemm_tn_persistent_kernel<BN, NSTG>, dim3(blocks), dim3(TCP_THREADS), smem, st, ma, mb, md, p, tiles_n, total);
    return true;
}
// FTP_TC_PERSIST=0: every product on the one-tile-per-block kernel (A/B measurements)
static bool persist_enabled() {
    static int on = -1;
    if (on < 0) { const char* e = std::getenv("FTP_TC_PERSIST"); on = (e && std::strcmp(e, "0") == 0) ? 0 : 1; }
    return on != 0;
}

// shared tail of the 1x1 and 3x3 launchers: plan, launch, second pass
template <int BN>
bool run_tn(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& md, TcParams p, float* scratch, cudaStream_t st) {
    const long long tiles = (long long)((p.N + BN - 1) / BN) * ((p.M + TC_BM - 1) / TC_BM);
    const int nkb = (p.K + TC_BK - 1) / TC_BK;
    TnPlan pl = plan_tn(tiles, nkb, (long long)p.M * p.N);
    if (!scratch || ((long long)p.M * p.N) % 4 != 0) { pl.S = 1; pl.kbps = nkb; }
    const __nv_bfloat16* addend = p.addend;
    if (pl.S > 1) { p.partial = scratch; p.kb_per_slice = pl.kbps; p.addend = nullptr; }
    if constexpr (BN == 64 || BN == 128) {
        // many tiles and a short reduction: the persistent kernel (its epilogues overlap the next tiles' loads).  Measured
        // on the 1x1 convolutions of MobileNetV2 at 224 x 224: 128-wide tiles 89 -> 70 us, 45 -> 40 us, 12.7 -> 8.3 us;
        // 32-wide tiles (direct stores, nothing to overlap) and the 3x3 convolutions of VGG-16 (nine or more reduction blocks
        // per tile: bound by bytes in flight from L2, which three resident blocks per SM hold more of) were slower.
        if (pl.S == 1 && tiles >= 2LL * sm_count() && !p.conv.enabled && nkb <= 4 && persist_enabled()) {
            if constexpr (BN == 128) return launch_tn_persistent<BN, 3>(ma, mb, md, p, st);       // 96 KB of ring beside 128 KB of staging tiles
            else return launch_tn_persistent<BN, 6>(ma, mb, md, p, st);
        }
    }
    const dim3 grid((p.N + BN - 1) / BN, (p.M + TC_BM - 1) / TC_BM, pl.S);
    bool ok;
    if constexpr (BN == 256) ok = launch_tn_kernel<BN, 4>(ma, mb, md, p, grid, st);              // 48 KB per stage: four fill the SM
    else ok = pl.stages == 6 ? launch_tn_kernel<BN, 6>(ma, mb, md, p, grid, st) : launch_tn_kernel<BN, 3>(ma, mb, md, p, grid, st);
    if (ok && pl.S > 1) {
        const long long count4 = (long long)p.M * p.N / 4;
        launch(slice_sum_bf16_kernel, dim3((unsigned)((count4 + 255) / 256)), dim3(256), 0, st, reinterpret_cast<const float4*>(scratch), pl.S, count4, addend, p.D);
    }
    return ok;
}

template <int BN>
bool launch_conv3x3(const __nv_bfloat16* A, const __nv_bfloat16* B, const __nv_bfloat16* addend, __nv_bfloat16* D, float* scratch, int N, int H, int W, int Ca,
                    int No, int flip, int* err, cudaStream_t st) {
    CUtensorMap ma, mb, md;
    if (!make_map_4d(&ma, A, N, H, W, Ca, TC_BM) || !make_map_2d(&mb, B, 9LL * No, Ca, BN)) return false;
    if (BN >= 64) { if (!make_map_2d(&md, D, (long long)N * H * W, No, TC_BM)) return false; }
    else md = mb;
    const int M = N * H * W;
    TcParams p{D, addend, M, No, 9 * Ca, err, ConvTap{1, H, W, Ca / 64, flip, No}, nullptr, 0};
    return run_tn<BN>(ma, mb, md, p, scratch, st);
}

template <int BN>
bool launch_tn(const __nv_bfloat16* A, const __nv_bfloat16* B, const __nv_bfloat16* addend, __nv_bfloat16* D, float* scratch, int M, int N, int K, int* err,
               cudaStream_t st) {
    CUtensorMap ma, mb, md;
    if (!make_map_2d(&ma, A, M, K, TC_BM) || !make_map_2d(&mb, B, N, K, BN)) return false;
    if (BN >= 64) { if (!make_map_2d(&md, D, M, N, TC_BM)) return false; }
    else md = mb;
    TcParams p{D, addend, M, N, K, err, ConvTap{0, 0, 0, 0, 0, 0}, nullptr, 0};
    return run_tn<BN>(ma, mb, md, p, scratch, st);
}

template <int BN>
bool launch_wgrad(const __nv_bfloat16* X, const __nv_bfloat16* dY, float* out, long long R, int Mo, int No, const TcWgPlan& w, int* err, cudaStream_t st) {
    CUtensorMap mx, my;
    if (!make_map_2d(&mx, X, R, Mo, 64) || !make_map_2d(&my, dY, R, No, 64)) return false;
    constexpr int smem = TC_STAGES * (2 + BN / 64) * 64 * 64 * 2 + 1024;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(tc_wgrad_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return false;
        configured = true;
    }
    TcWgParams p{out, Mo, No, (int)R, w.rows_per_split, err, ConvTap{0, 0, 0, 0, 0, 0}, 0};
    launch(tc_wgrad_kernel<BN>, dim3((Mo + TC_BM - 1) / TC_BM, (No + BN - 1) / BN, w.S), dim3(TC_THREADS), smem, st, mx, my, p);
    return true;
}

template <int BN>
bool launch_wgrad3x3(const __nv_bfloat16* X, const __nv_bfloat16* dY, float* out, int N, int H, int W, int Mo, int No, const TcWgPlan& w, int* err,
                     cudaStream_t st) {
    CUtensorMap mx, my;
    const long long R = (long long)N * H * W;
    if (!make_map_4d(&mx, X, N, H, W, Mo, 64) || !make_map_2d(&my, dY, R, No, 64)) return false;
    constexpr int smem = TC_STAGES * (2 + BN / 64) * 64 * 64 * 2 + 1024;
    if (cudaFuncSetAttribute(tc_wgrad_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return false;
    const int pair = wgrad3x3_pairs_taps(Mo) ? 1 : 0;
    TcWgParams p{out, Mo, No, (int)R, w.rows_per_split, err, ConvTap{1, H, W, 0, 0, 0}, pair};
    launch(tc_wgrad_kernel<BN>, dim3((Mo + TC_BM - 1) / TC_BM, (No + BN - 1) / BN, w.S * (pair ? 5 : 9)), dim3(TC_THREADS), smem, st, mx, my, p);
    return true;
}

TcWgPlan plan_tc_wgrad3x3(long long R, int Mo, int No) {
    const long long tiles = (wgrad3x3_pairs_taps(Mo) ? 5LL : 9LL) * ((Mo + TC_BM - 1) / TC_BM) * ((No + 127) / 128);
    long long S = (2LL * sm_count() + tiles - 1) / tiles;
    // tiles that already cover about half of the SMs take the whole reduction each and write dW directly: the float
    // partial sums of these layers are as large as the weights (9 x 512 x 512), and writing and re-reading two or three
    // copies of them cost more than the second wave of blocks saved (VGG-16 at batch 256: 1.484 -> 1.400 ms per step;
    // the same rule from a fifth of the SMs on: 1.516 ms)
    if (tiles * 100 >= 45LL * sm_count()) S = 1;
    const long long maxS = (R + 511) / 512;
    long long cap = (8LL << 20) / (9LL * Mo * No);
    if (cap < 1) cap = 1;
    if (S > maxS) S = maxS;
    if (S > cap) S = cap;
    if (S < 1) S = 1;
    const long long rps = ((R + S - 1) / S + 63) / 64 * 64;
    TcWgPlan w;
    w.rows_per_split = (int)rps;
    w.S = (int)((R + rps - 1) / rps);
    return w;
}

}  // namespace

bool tc_conv3x3_supported(int N, int H, int W, int Ca, int No, const void* A, const void* B, const void* D, const void* addend) {
    auto a16 = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; };
    return Ca % 64 == 0 && No % 8 == 0 && conv_tiles_ok(H, W, TC_BM) && conv_tiles_ok(H, W, 64) && (long long)N * H * W < (1LL << 31) && a16(A) &&
           a16(B) && a16(D) && a16(addend) && encode_fn() != nullptr;
}

// 3x3, stride 1, pad 1.  Forward (flip 0): A = x (N,H,W,Ca), B = weights [9][No][Ca]; data gradient (flip 1): A = dy,
// B = weights [9][No = cin][Ca = cout].  D (N,H,W,No) bf16.
bool tc_conv3x3(const __nv_bfloat16* A, const __nv_bfloat16* B, const __nv_bfloat16* addend, __nv_bfloat16* D, float* scratch, int N, int H, int W, int Ca,
                int No, int flip, int* err, cudaStream_t st) {
    if (use_bn256(N * H * W, No, 9 * Ca)) return launch_conv3x3<256>(A, B, addend, D, scratch, N, H, W, Ca, No, flip, err, st);
    if (No > 64) return launch_conv3x3<128>(A, B, addend, D, scratch, N, H, W, Ca, No, flip, err, st);
    if (No > 32) return launch_conv3x3<64>(A, B, addend, D, scratch, N, H, W, Ca, No, flip, err, st);
    return launch_conv3x3<32>(A, B, addend, D, scratch, N, H, W, Ca, No, flip, err, st);
}

size_t tc_gemm_scratch_floats(int M, int N, int K) {
    size_t most = 0;
    for (int BN : {32, 64, 128, 256}) {
        const long long tiles = (long long)((N + BN - 1) / BN) * ((M + TC_BM - 1) / TC_BM);
        const TnPlan pl = plan_tn(tiles, (K + TC_BK - 1) / TC_BK, (long long)M * N);
        if (pl.S > 1) most = std::max(most, (size_t)pl.S * M * N);
    }
    return most;
}

size_t tc_wgrad3x3_scratch_floats(long long R, int Mo, int No) {
    const TcWgPlan w = plan_tc_wgrad3x3(R, Mo, No);
    return w.S > 1 ? (size_t)w.S * 9 * Mo * No : 0;
}

// dW[9][Mo][No] of a 3x3 / stride 1 / pad 1 convolution; returns the number of splits (0: nothing launched)
int tc_wgrad3x3(const __nv_bfloat16* X, const __nv_bfloat16* dY, float* dW, float* scratch, int N, int H, int W, int Mo, int No, int* err, cudaStream_t st) {
    const TcWgPlan w = plan_tc_wgrad3x3((long long)N * H * W, Mo, No);
    float* out = w.S > 1 ? scratch : dW;
    const bool ok = No > 64 ? launch_wgrad3x3<128>(X, dY, out, N, H, W, Mo, No, w, err, st) : launch_wgrad3x3<64>(X, dY, out, N, H, W, Mo, No, w, err, st);
    return ok ? w.S : 0;
}

size_t tc_wgrad_scratch_floats(long long R, int Mo, int No) {
    const TcWgPlan w = plan_tc_wgrad(R, Mo, No);
    return w.S > 1 ? (size_t)w.S * Mo * No : 0;
}

// dW[Mo][No] = X[R][Mo]^T * dY[R][No] (bf16 in, float out); scratch holds tc_wgrad_scratch_floats floats.
// Returns the number of splits written to scratch (1: dW was written directly), 0 if nothing was launched.
int tc_wgrad(const __nv_bfloat16* X, const __nv_bfloat16* dY, float* dW, float* scratch, long long R, int Mo, int No, int* err, cudaStream_t st) {
    const TcWgPlan w = plan_tc_wgrad(R, Mo, No);
    float* out = w.S > 1 ? scratch : dW;
    const bool ok = No > 64 ? launch_wgrad<128>(X, dY, out, R, Mo, No, w, err, st) : launch_wgrad<64>(X, dY, out, R, Mo, No, w, err, st);
    return ok ? w.S : 0;
}

bool tc_gemm_supported(int M, int N, int K, const void* A, const void* B, const void* D, const void* addend) {
    auto a16 = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; };
    return M >= 1 && N % 8 == 0 && K % 8 == 0 && N >= 8 && K >= 8 && a16(A) && a16(B) && a16(D) && a16(addend) && encode_fn() != nullptr;
}

bool tc_gemm_tn(const __nv_bfloat16* A, const __nv_bfloat16* B, const __nv_bfloat16* addend, __nv_bfloat16* D, float* scratch, int M, int N, int K, int* err,
                cudaStream_t st) {
    if (use_bn256(M, N, K)) return launch_tn<256>(A, B, addend, D, scratch, M, N, K, err, st);
    if (N > 64) return launch_tn<128>(A, B, addend, D, scratch, M, N, K, err, st);
    if (N > 32) return launch_tn<64>(A, B, addend, D, scratch, M, N, K, err, st);
    return launch_tn<32>(A, B, addend, D, scratch, M, N, K, err, st);
}

}  // namespace ftp
