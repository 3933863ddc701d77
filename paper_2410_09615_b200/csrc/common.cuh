// Shared device/host helpers of libslim (CUDA side only).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "slim.h"

namespace slim {

// Bit a device-detected error sets in the caller's status word.
__device__ __forceinline__ void flag_error(uint32_t* status_dev, int code) {
    if (status_dev) atomicOr(status_dev, 1u << code);
}

__host__ __device__ __forceinline__ int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Per-device facts the launchers need (filled once per device, read-only after).
struct DeviceInfo {
    int cc_major;
    int sm_count;
    int decode_ctas_per_sm[2];   // cooperative residency of the decode kernel, NT = 1, 2
    int decode_tiled_ok;         // every variant of the tiled decode kernel can be resident once per SM
};
const DeviceInfo* device_info(slim_status_t* err);

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda);
// nullptr when the driver does not have it.  Thread-safe.
void* tensor_map_encoder();

// The decode kernels keep the published T = X R^T at the start of the workspace, in a region of
// this fixed size, so that calls of different shapes and kernels never read one kind of slot as another.
constexpr size_t kDecodeTfinalBytes = 198656;

// Launch bookkeeping for slim_last_launch_count().
void count_launch(int n);
void reset_launch_count();
void note_token_tile(int n);      // token-tile width of the prefill main launch, for slim_last_token_tile()

// ---- launchers (defined in the kernel files) --------------------------------
slim_status_t launch_pack(const int8_t* codes, const uint8_t* mask, int d_out, int d_in,
                          uint8_t* vals, uint8_t* meta, uint32_t* status_dev, cudaStream_t st);
slim_status_t launch_unpack(const uint8_t* vals, const uint8_t* meta, int d_out, int d_in,
                            int8_t* codes, uint8_t* mask, cudaStream_t st);

size_t simple_workspace_bytes(int b, int d_out, int d_in, int r);
slim_status_t launch_simple(const __nv_bfloat16* X, int b, const uint8_t* vals, const uint8_t* meta,
                            float s, const __nv_bfloat16* L, const __nv_bfloat16* R, int r,
                            int d_out, int d_in, __nv_bfloat16* Y, void* ws, cudaStream_t st);

bool decode_supports(int b, int d_out, int d_in, int r);
size_t decode_workspace_bytes(int b, int d_out, int d_in, int r);
slim_status_t launch_decode(const __nv_bfloat16* X, int b, const uint8_t* vals, const uint8_t* meta,
                            float s, const __nv_bfloat16* L, const __nv_bfloat16* R, int r,
                            int d_out, int d_in, __nv_bfloat16* Y, void* ws, uint32_t* status_dev,
                            cudaStream_t st);
bool decode_supports_q(int b, int d_out, int d_in, int r);
slim_status_t launch_decode_q(const __nv_bfloat16* X, int b, const uint8_t* vals, const uint8_t* meta, float s,
                              const uint8_t* Lq, const __nv_bfloat16* Ls, const uint8_t* Rq, const __nv_bfloat16* Rs, int r,
                              int d_out, int d_in, __nv_bfloat16* Y, void* ws, uint32_t* status_dev, cudaStream_t st);
int decode_query_residency(int nt);

bool decode_tiled_supports(int b, int d_out, int d_in, int r);
size_t decode_tiled_workspace_bytes(int b, int d_out, int d_in, int r);
slim_status_t launch_decode_tiled(const __nv_bfloat16* X, int b, const uint8_t* W, float s, const __nv_bfloat16* L,
                                  const __nv_bfloat16* R, int r, int d_out, int d_in, __nv_bfloat16* Y, void* ws,
                                  uint32_t* status_dev, cudaStream_t st);
int decode_tiled_query_residency();

slim_status_t launch_repack_tiled(const uint8_t* vals, const uint8_t* meta, int d_out, int d_in, uint8_t* out, cudaStream_t st);

slim_status_t launch_pack_adapter(const __nv_bfloat16* A, int rows, int cols, uint8_t* codes, __nv_bfloat16* scales, cudaStream_t st);
slim_status_t launch_unpack_adapter(const uint8_t* codes, const __nv_bfloat16* scales, int rows, int cols, __nv_bfloat16* out,
                                    cudaStream_t st);

slim_status_t launch_mask_top2(const int8_t* codes, const float* xbar, int d_out, int d_in, uint8_t* mask, uint32_t* status_dev,
                               cudaStream_t st);
size_t quant_workspace_bytes(int d_out, int d_in);
slim_status_t launch_quant(const float* W, int d_out, int d_in, int8_t* codes, float* scale_alpha, void* ws,
                           uint32_t* status_dev, cudaStream_t st);

bool prefill_supports(int b, int d_out, int d_in, int r);
size_t prefill_workspace_bytes(int b, int d_out, int d_in, int r);
slim_status_t launch_prefill(const __nv_bfloat16* X, int b, const uint8_t* vals, const uint8_t* meta,
                             float s, const __nv_bfloat16* L, const __nv_bfloat16* R, int r,
                             int d_out, int d_in, __nv_bfloat16* Y, void* ws, uint32_t* status_dev,
                             cudaStream_t st, bool force_pair = false);

}  // namespace slim
