// Quantized adapters (Sec. 3.3 "Low-rank Adapter Quantization": 4-bit AbsMax, groups of 128 elements
// share one parameter).  Storage and arithmetic as include/slim.h states them: a group is 128
// consecutive elements of a row (rows run along the contraction axis), its bf16 scale is absmax / 7
// (binary32 division, nearest-even to bf16), a code is clamp(rint(a / scale), -8, 7) with the division
// in binary32, two codes per byte (even column in the low nibble).
#include "common.cuh"

namespace slim {

// One warp per (row, group): a lane holds four consecutive elements.
__global__ void pack_adapter_kernel(const __nv_bfloat16* __restrict__ A, int rows, int cols, int groups,
                                    uint8_t* __restrict__ codes, __nv_bfloat16* __restrict__ scales)
{
    const int lane = threadIdx.x & 31;
    const long long item = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (item >= (long long)rows * groups) return;
    const int row = (int)(item / groups), grp = (int)(item % groups);
    const int c0 = grp * 128 + lane * 4;
    float v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = c0 + i < cols ? __bfloat162float(A[(size_t)row * cols + c0 + i]) : 0.f;
    float m = fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3])));
#pragma unroll
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    const __nv_bfloat16 sb = m > 0.f ? __float2bfloat16_rn(__fdiv_rn(m, 7.0f)) : __float2bfloat16_rn(0.f);
    const float sc = __bfloat162float(sb);
    if (lane == 0) scales[(size_t)row * groups + grp] = sb;
    uint32_t q[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int c = 0;
        if (sc > 0.f) c = max(-8, min(7, __float2int_rn(__fdiv_rn(v[i], sc))));     // nearest, ties to even
        q[i] = (uint32_t)c & 0xFu;
    }
    // cols is even, so elements come in pairs: either both of a byte exist or neither
    uint8_t* dst = codes + (size_t)row * (cols / 2) + c0 / 2;
    if (c0 + 3 < cols) *reinterpret_cast<uint16_t*>(dst) = (uint16_t)(q[0] | (q[1] << 4) | (q[2] << 8) | (q[3] << 12));
    else if (c0 + 1 < cols) dst[0] = (uint8_t)(q[0] | (q[1] << 4));
}

// One thread per byte of codes: two bf16 values out.
__global__ void unpack_adapter_kernel(const uint8_t* __restrict__ codes, const __nv_bfloat16* __restrict__ scales, int rows,
                                      int cols, int groups, __nv_bfloat16* __restrict__ out)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t half = (size_t)cols / 2;
    if (i >= (size_t)rows * half) return;
    const int row = (int)(i / half), c = 2 * (int)(i % half);
    const float sc = __bfloat162float(scales[(size_t)row * groups + c / 128]);
    const uint32_t B = codes[i];
    const int lo = (int)(B & 0xFu), hi = (int)(B >> 4);
    const float a = (float)(lo >= 8 ? lo - 16 : lo) * sc, b = (float)(hi >= 8 ? hi - 16 : hi) * sc;
    *reinterpret_cast<__nv_bfloat162*>(out + (size_t)row * cols + c) = __floats2bfloat162_rn(a, b);
}

slim_status_t launch_pack_adapter(const __nv_bfloat16* A, int rows, int cols, uint8_t* codes, __nv_bfloat16* scales, cudaStream_t st)
{
    const int groups = (cols + 127) / 128;
    const long long items = (long long)rows * groups;
    pack_adapter_kernel<<<(unsigned)((items + 7) / 8), 256, 0, st>>>(A, rows, cols, groups, codes, scales);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

slim_status_t launch_unpack_adapter(const uint8_t* codes, const __nv_bfloat16* scales, int rows, int cols, __nv_bfloat16* out,
                                    cudaStream_t st)
{
    const size_t n = (size_t)rows * (cols / 2);
    unpack_adapter_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(codes, scales, rows, cols, (cols + 127) / 128, out);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

}  // namespace slim
