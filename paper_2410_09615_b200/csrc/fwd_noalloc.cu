// slim_linear_fwd_noalloc: the small-batch forward for callers that may not
// allocate device memory.  Its scratch lives in this file's static device
// array; everything else is the ordinary decode kernel.
#include <mutex>
#include "common.cuh"

namespace slim {

// Scratch shared by every call of slim_linear_fwd_noalloc on a device: split-K
// partial slots plus, in its first SLIM_WORKSPACE_SYNC_BYTES, the call counter.  Each GPU that loads the library carries one copy until exit.
static __device__ __align__(256) unsigned char g_noalloc_scratch[SLIM_NOALLOC_SCRATCH_BYTES];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an
// address the GPU can use; the device address is looked up once per device.
static void* g_scratch_addr[64];
static std::mutex g_scratch_mutex;

static slim_status_t scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SLIM_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return SLIM_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return SLIM_OK;
}

static bool is_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace slim

using namespace slim;

extern "C" size_t slim_noalloc_scratch_needed(int b, int d_out, int d_in, int r)
{
    if (b < 1 || b > 16 || r < 0 || d_out < 1 || d_in < 1 || d_in % 64 != 0 || d_out % 16 != 0 || r % 16 != 0) return 0;
    const size_t need = decode_workspace_bytes(b, d_out, d_in, r);
    return need ? SLIM_WORKSPACE_SYNC_BYTES + need : 0;
}

extern "C" slim_status_t slim_linear_fwd_noalloc(const void* X, int b, const uint8_t* vals,
                                                 const uint8_t* meta, float s, const void* L,
                                                 const void* R, int r, int d_out, int d_in, void* Y,
                                                 uint32_t* status_dev, void* cuda_stream)
{
    reset_launch_count();
    if (!X || !vals || !meta || !Y || b < 1 || r < 0 || d_out < 1 || d_in < 1) return SLIM_ERR_INVALID_ARG;
    if ((r > 0) != (L != nullptr) || (r > 0) != (R != nullptr)) return SLIM_ERR_INVALID_ARG;
    if (d_in % 64 != 0 || d_out % 16 != 0 || r % 16 != 0) return SLIM_ERR_UNSUPPORTED_SHAPE;
    if (!is_aligned16(X) || !is_aligned16(vals) || !is_aligned16(meta) || !is_aligned16(Y) || !is_aligned16(L) ||
        !is_aligned16(R))
        return SLIM_ERR_INVALID_ARG;
    if (status_dev && (reinterpret_cast<uintptr_t>(status_dev) & 3u)) return SLIM_ERR_INVALID_ARG;
    // only problems the decode kernel takes, and only while its scratch fits the static array
    const size_t need = decode_workspace_bytes(b, d_out, d_in, r);
    if (b > 16 || need == 0) return SLIM_ERR_UNSUPPORTED_SHAPE;
    if (SLIM_WORKSPACE_SYNC_BYTES + need > (size_t)SLIM_NOALLOC_SCRATCH_BYTES) return SLIM_ERR_WORKSPACE;
    slim_status_t derr;
    if (!device_info(&derr)) return derr;
    if (!decode_supports(b, d_out, d_in, r)) return SLIM_ERR_UNSUPPORTED_SHAPE;
    void* scratch = nullptr;
    slim_status_t st = scratch_address(&scratch);
    if (st != SLIM_OK) return st;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // the array keeps whatever the previous call left (possibly of another shape, possibly cut
    // short by a timeout): mark this call's hand-over slots empty and restart the call counter
    if (cudaMemsetAsync(static_cast<char*>(scratch) + SLIM_WORKSPACE_SYNC_BYTES, 0xFF, need, stream) != cudaSuccess ||
        cudaMemsetAsync(scratch, 0, SLIM_WORKSPACE_SYNC_BYTES, stream) != cudaSuccess)
        return SLIM_ERR_CUDA;
    return launch_decode(static_cast<const __nv_bfloat16*>(X), b, vals, meta, s,
                         static_cast<const __nv_bfloat16*>(L), static_cast<const __nv_bfloat16*>(R), r, d_out,
                         d_in, static_cast<__nv_bfloat16*>(Y), scratch, status_dev, stream);
}
