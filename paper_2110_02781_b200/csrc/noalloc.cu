// Weight gradient of a dense convolution for callers that must not allocate device memory.
//
// The split reduction of the weight-gradient kernel needs a scratch area for its partial sums.
// Everywhere else in this library the caller supplies that memory inside the model workspace.
// Some callers cannot: code running inside a region where cudaMalloc is forbidden or would
// synchronise the device (a stream-ordered pipeline that must not stall, a plug-in whose host
// gives it input and output buffers and nothing else, a process whose memory pool is owned by
// another component).  For them the scratch lives in a fixed-size array in the library's own
// device image; every GPU that loads the library carries it until the process exits.
#include <atomic>
#include <cstdint>
#include "common.h"
#include "kernels.h"

namespace {

constexpr size_t kScratchFloats = size_t(1) << 21;          // 8 MiB: the stated, modest maximum
static __device__ __align__(256) float g_wgrad_scratch[kScratchFloats];

constexpr int kMaxDevices = 64;
std::atomic<float*> g_scratch_addr[kMaxDevices] = {};       // device address of the array, per device (every thread that looks it up gets the same value)

// In host code the array's name is only a handle; the address a kernel may use has to be asked
// for, once per device, with that device current.
ftp_status scratch_for_current_device(float** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return ftp::fail(FTP_ECUDA, "conv_wgrad_static: cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return ftp::fail(FTP_ERANGE, "conv_wgrad_static: device index %d not supported", dev);
    float* addr = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!addr) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_wgrad_scratch);
        if (e != cudaSuccess || !p) return ftp::fail(FTP_ECUDA, "conv_wgrad_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        addr = static_cast<float*>(p);
        g_scratch_addr[dev].store(addr, std::memory_order_release);
    }
    *out = addr;
    return FTP_OK;
}

}  // namespace

extern "C" ftp_status ftp_conv_wgrad_static(const float* x, const float* dy, float* dw, int32_t n, int32_t h, int32_t w,
                                            int32_t cin, int32_t cout, int32_t k, int32_t stride, int32_t pad, void* stream) {
    FTP_REQUIRE(x && dy && dw, FTP_EINVAL, "conv_wgrad_static: null buffer");
    FTP_REQUIRE(n >= 1 && h >= 1 && w >= 1 && cin >= 1 && cout >= 1 && k >= 1 && stride >= 1 && pad >= 0, FTP_EINVAL,
                "conv_wgrad_static: sizes must be positive");
    FTP_REQUIRE(h + 2 * pad >= k && w + 2 * pad >= k, FTP_EINVAL, "conv_wgrad_static: kernel larger than the padded input");
    // the kernels index the filter with int: k*k*cin (the reduction length) and k*k*cin*cout (the size of dw) must fit
    FTP_REQUIRE((long long)k * k * cin < (1LL << 31) && (long long)k * k * cin * cout < (1LL << 31), FTP_ERANGE,
                "conv_wgrad_static: filter too large (k*k*cin*cout must stay below 2^31)");
    ftp::ConvGeom g{n, h, w, cin, (h + 2 * pad - k) / stride + 1, (w + 2 * pad - k) / stride + 1, cout, k, k, stride, pad, pad};
    FTP_REQUIRE((long long)n * h * w * cin < (1LL << 31) && (long long)n * g.Ho * g.Wo * cout < (1LL << 31), FTP_ERANGE,
                "conv_wgrad_static: tensor too large");
    const size_t need = ftp::conv_wgrad_scratch_floats(g);
    FTP_REQUIRE(need <= kScratchFloats, FTP_ERANGE,
                "conv_wgrad_static: this shape needs %zu floats of scratch, the built-in area holds %zu; use the model API", need,
                kScratchFloats);
    float* scratch = nullptr;
    ftp_status s = scratch_for_current_device(&scratch);
    if (s != FTP_OK) return s;
    // Every partial the second pass reads is written by the first pass of the same call, so nothing
    // left over from an earlier call has to be cleared.
    ftp::conv_wgrad_f32(x, dy, dw, scratch, g, static_cast<cudaStream_t>(stream));
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return ftp::fail(FTP_ECUDA, "conv_wgrad_static: launch failed: %s", cudaGetErrorString(e));
    return FTP_OK;
}
