// dmr_lowbit_linear_noalloc: the decode-time low-bit linear layer for callers that cannot give the
// library a workspace because they cannot allocate device memory at the point of the call - a
// serving loop that handed all free memory to its cache pool at start-up, or a plug-in that runs
// inside another program's step and is not allowed to touch its allocator (cudaMalloc may also
// synchronise the whole device, which such a loop cannot afford).  The scratch the streaming kernel
// needs lives in a fixed array inside the library image instead.
#include <mutex>

#include "common.cuh"

namespace dmr {

namespace {

// Limits of the fixed scratch: enough for N <= kNoallocMaxN output features on a GPU with up to
// kMaxStreamCtas / 2 SMs.  Every GPU that loads the library holds this array until the process exits.
constexpr int kNoallocMaxN = 65536;
constexpr size_t kNoallocStatusBytes = 256;
constexpr size_t kNoallocScratchBytes =
    kNoallocStatusBytes + kStreamPartialBytes + (size_t)(kNoallocMaxN / 128) * kCounterStride * sizeof(int32_t);

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoallocScratchBytes];

std::mutex g_setup_mutex;
void *g_scratch_on_device[64] = {};  // device address of the array, per device ordinal

// Looks up (once per device, with that device current) where the array lives on the device.
dmr_status_t scratch_address(void **out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= 64) {
        g_last_cuda_error = (int)(e != cudaSuccess ? e : cudaErrorInvalidDevice);
        return DMR_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_on_device[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) {
            g_last_cuda_error = (int)e;
            (void)cudaGetLastError();
            return DMR_ERR_CUDA;
        }
        g_scratch_on_device[dev] = p;
    }
    *out = g_scratch_on_device[dev];
    return DMR_OK;
}

}  // namespace
}  // namespace dmr

using namespace dmr;

extern "C" {

int dmr_noalloc_max_n(void) { return kNoallocMaxN; }

dmr_status_t dmr_lowbit_linear_noalloc(const void *X_bf16, int M, const void *qweight, const void *scales,
                                       const void *zeros, int N, int K, dmr_qformat_t f, void *Y, dmr_out_t out,
                                       void *stream) {
    if (M < 0 || N < 1 || K < 1) return DMR_ERR_INVALID_ARG;
    if (out != DMR_OUT_BF16 && out != DMR_OUT_F32) return DMR_ERR_INVALID_ARG;
    if (M > 0 && (!X_bf16 || !Y)) return DMR_ERR_INVALID_ARG;
    if (!qweight || !scales || !zeros) return DMR_ERR_INVALID_ARG;
    if (f.bits != 4 && f.bits != 8) return DMR_ERR_UNSUPPORTED;
    if (!format_ok(K, f)) return DMR_ERR_INVALID_ARG;
    if (!aligned16(X_bf16) || !aligned16(Y) || !aligned16(qweight)) return DMR_ERR_ALIGNMENT;
    // beyond the fixed scratch, or a shape only the workspace-taking entry point has kernels for
    if (M > 16 || N > kNoallocMaxN || !stream_supported(M == 0 ? 1 : M, N, K, f.bits, group_of(K, f))) return DMR_ERR_UNSUPPORTED;
    if (M == 0) return DMR_OK;
    void *base = nullptr;
    dmr_status_t r = scratch_address(&base);
    if (r != DMR_OK) return r;
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps what the last call left: the status word must start at zero (the kernel leaves
    // its counters at zero itself)
    cudaError_t e = cudaMemsetAsync(base, 0, kNoallocStatusBytes, st);
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        return DMR_ERR_CUDA;
    }
    RowSel sel = {nullptr, nullptr, 0};
    return launch_stream(reinterpret_cast<const uint16_t *>(X_bf16), M, sel, qweight, reinterpret_cast<const uint16_t *>(scales),
                         reinterpret_cast<const uint8_t *>(zeros), N, K, f.bits, group_of(K, f), Y, out,
                         reinterpret_cast<char *>(base) + kNoallocStatusBytes, reinterpret_cast<int32_t *>(base), st);
}

}  // extern "C"
