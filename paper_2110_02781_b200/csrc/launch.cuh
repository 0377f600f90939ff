// Kernel launches with programmatic dependent launch: a kernel may be scheduled while the kernel before it on
// the stream is still draining, so that launch latency and the set-up part of a block overlap the tail of the
// predecessor.  Every kernel launched through `launch` calls grid_dep_sync() before it touches global memory:
// that wait returns only when the whole preceding grid has completed and its writes are visible, so the
// ordering of memory effects is the same as with plain stream order.
#pragma once
#include <cuda_runtime.h>
#include <utility>

namespace ftp {

__device__ __forceinline__ void grid_dep_sync() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
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
    cudaLaunchKernelEx(&cfg, kern, std::forward<A>(args)...);
}

}  // namespace ftp
