// Kernel launches with programmatic dependent launch: a kernel may be scheduled while the kernel before it on
// the stream is still draining, so that launch latency and the set-up part of a block overlap the tail of the
// predecessor.  Every kernel launched through `launch` calls grid_dep_sync() before it touches global memory:
// that wait returns only when the whole preceding grid has completed and its writes are visible, so the
// ordering of memory effects is the same as with plain stream order.
#pragma once
#include <cuda_runtime.h>
#include <utility>
#ifdef FTP_TIMELINE
#include <vector>
#endif

namespace ftp {

#ifdef FTP_TIMELINE
// Measurement build only (-DFTP_TIMELINE): the first thread of every grid notes the time at which its wait on the
// preceding grid returned.  On one stream those times are in launch order, so the gap to the next entry is what the
// launch costs in a replayed step, with no events in between.  Every translation unit has its own buffer; the
// buffers are merged by time on the host (ftp_debug_timeline).
constexpr unsigned TL_CAP = 1u << 15;
static __device__ unsigned long long g_tl_time[2 * TL_CAP];     // per entry: the time, then the grid's signature (tl_signature)
static __device__ unsigned g_tl_count;
void tl_register(void (*reader)(std::vector<unsigned long long>&, bool));
// host side: the kernels in launch order with their signature and stream, for naming the entries (with two streams the
// grids start in another order than they were launched: an entry is the k-th launch of its signature)
void tl_note_launch(const void* kernel, unsigned long long signature, const void* stream);
__host__ __device__ inline unsigned long long tl_signature(unsigned gx, unsigned gy, unsigned gz, unsigned threads) {
    return (unsigned long long)gx | (unsigned long long)gy << 24 | (unsigned long long)gz << 40 | (unsigned long long)threads << 52;
}
static void tl_reader(std::vector<unsigned long long>& out, bool reset) {
    unsigned n = 0;
    if (cudaMemcpyFromSymbol(&n, g_tl_count, sizeof n) != cudaSuccess) return;
    if (n > TL_CAP) n = TL_CAP;
    const size_t at = out.size();
    out.resize(at + 2 * (size_t)n);
    if (n) cudaMemcpyFromSymbol(out.data() + at, g_tl_time, 2 * (size_t)n * sizeof(unsigned long long));
    if (reset) { const unsigned z = 0; cudaMemcpyToSymbol(g_tl_count, &z, sizeof z); }
}
namespace { struct TlRegistrar { TlRegistrar() { tl_register(&tl_reader); } } g_tl_registrar; }
#endif

__device__ __forceinline__ void grid_dep_sync() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
#ifdef FTP_TIMELINE
    if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0 && threadIdx.y == 0 && threadIdx.z == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        const unsigned i = atomicAdd(&g_tl_count, 1u);
        if (i < TL_CAP) { g_tl_time[2 * i] = t; g_tl_time[2 * i + 1] = tl_signature(gridDim.x, gridDim.y, gridDim.z, blockDim.x * blockDim.y * blockDim.z); }
    }
#endif
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

bool pdl_enabled();     // false when the environment sets FTP_PDL=0

template <typename... KA, typename... A>
inline void launch(void (*kern)(KA...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, A&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
#ifdef FTP_TIMELINE
    tl_note_launch(reinterpret_cast<const void*>(kern), tl_signature(grid.x, grid.y, grid.z, block.x * block.y * block.z), st);
#endif
    cudaLaunchKernelEx(&cfg, kern, std::forward<A>(args)...);
}

}  // namespace ftp
