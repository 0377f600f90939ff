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
static __device__ unsigned long long g_tl_time[TL_CAP];
static __device__ unsigned g_tl_count;
void tl_register(void (*reader)(std::vector<unsigned long long>&, bool));
void tl_note_launch(const void* kernel);            // host side: the kernels in launch order, for naming the entries
static void tl_reader(std::vector<unsigned long long>& out, bool reset) {
    unsigned n = 0;
    if (cudaMemcpyFromSymbol(&n, g_tl_count, sizeof n) != cudaSuccess) return;
    if (n > TL_CAP) n = TL_CAP;
    const size_t at = out.size();
    out.resize(at + n);
    if (n) cudaMemcpyFromSymbol(out.data() + at, g_tl_time, n * sizeof(unsigned long long));
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
        if (i < TL_CAP) g_tl_time[i] = t;
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
    tl_note_launch(reinterpret_cast<const void*>(kern));
#endif
    cudaLaunchKernelEx(&cfg, kern, std::forward<A>(args)...);
}

}  // namespace ftp
