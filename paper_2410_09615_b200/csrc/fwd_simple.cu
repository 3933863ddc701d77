// CUDA-core forward for any legal shape: the on-GPU correctness anchor and the
// dispatcher's path for shapes the tensor-core kernels do not take.
//   kernel 1: T[m][j] = sum_k X[m][k] R[j][k]            (fp32, into the workspace)
//   kernel 2: Y[m][n] = s * sum_kept X[m][k] q[n][k] + sum_j T[m][j] L[n][j]
// One warp per output element, lanes stride the contraction axis, shuffle reduce.
#include "common.cuh"

namespace slim {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__global__ void __launch_bounds__(256)
simple_t_kernel(const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ R,
                int b, int r, int d_in, float* __restrict__ T)
{
    const int lane = threadIdx.x & 31;
    const long long total = (long long)b * r;
    for (long long o = blockIdx.x * 8LL + (threadIdx.x >> 5); o < total; o += gridDim.x * 8LL) {
        const int m = (int)(o / r), j = (int)(o % r);
        const __nv_bfloat162* xr = reinterpret_cast<const __nv_bfloat162*>(X + (size_t)m * d_in);
        const __nv_bfloat162* rr = reinterpret_cast<const __nv_bfloat162*>(R + (size_t)j * d_in);
        float acc = 0.f;
        for (int k = lane; k < d_in / 2; k += 32) {
            const float2 a = __bfloat1622float2(xr[k]);
            const float2 c = __bfloat1622float2(rr[k]);
            acc = fmaf(a.x, c.x, acc);
            acc = fmaf(a.y, c.y, acc);
        }
        acc = warp_sum(acc);
        if (lane == 0) T[o] = acc;
    }
}

__global__ void __launch_bounds__(256)
simple_y_kernel(const __nv_bfloat16* __restrict__ X, const uint8_t* __restrict__ vals,
                const uint8_t* __restrict__ meta, float s, const __nv_bfloat16* __restrict__ L,
                const float* __restrict__ T, int b, int r, int d_out, int d_in,
                __nv_bfloat16* __restrict__ Y)
{
    const int lane = threadIdx.x & 31;
    const long long total = (long long)b * d_out;
    const int groups = d_in / 4;
    for (long long o = blockIdx.x * 8LL + (threadIdx.x >> 5); o < total; o += gridDim.x * 8LL) {
        const int m = (int)(o / d_out), n = (int)(o % d_out);
        const __nv_bfloat16* xr = X + (size_t)m * d_in;
        const uint8_t* vr = vals + (size_t)n * groups;
        const uint8_t* mr = meta + (size_t)n * (d_in / 8);
        float acc = 0.f;
        for (int g = lane; g < groups; g += 32) {
            const uint32_t vb = vr[g];
            const uint32_t mt = (mr[g >> 1] >> (4 * (g & 1))) & 0xFu;
            const int c0 = ((int)((vb & 0xFu) << 28)) >> 28;
            const int c1 = ((int)((vb >> 4) << 28)) >> 28;
            acc = fmaf(__bfloat162float(xr[4 * g + (mt & 3)]), (float)c0, acc);
            acc = fmaf(__bfloat162float(xr[4 * g + (mt >> 2)]), (float)c1, acc);
        }
        acc = warp_sum(acc) * s;
        float lr = 0.f;
        for (int j = lane; j < r; j += 32)
            lr = fmaf(T[(size_t)m * r + j], __bfloat162float(L[(size_t)n * r + j]), lr);
        lr = warp_sum(lr);
        if (lane == 0) Y[o] = __float2bfloat16_rn(acc + lr);
    }
}

size_t simple_workspace_bytes(int b, int d_out, int d_in, int r) {
    (void)d_out; (void)d_in;
    return (size_t)b * (size_t)r * sizeof(float);
}

slim_status_t launch_simple(const __nv_bfloat16* X, int b, const uint8_t* vals, const uint8_t* meta,
                            float s, const __nv_bfloat16* L, const __nv_bfloat16* R, int r,
                            int d_out, int d_in, __nv_bfloat16* Y, void* ws, cudaStream_t st)
{
    slim_status_t err;
    const DeviceInfo* di = device_info(&err);
    if (!di) return err;
    float* T = reinterpret_cast<float*>(reinterpret_cast<char*>(ws) + SLIM_WORKSPACE_SYNC_BYTES);
    const int cap = di->sm_count * 16;
    if (r > 0) {
        long long blocks = ((long long)b * r + 7) / 8;
        simple_t_kernel<<<(int)(blocks < cap ? blocks : cap), 256, 0, st>>>(X, R, b, r, d_in, T);
        count_launch(1);
    }
    long long blocks = ((long long)b * d_out + 7) / 8;
    simple_y_kernel<<<(int)(blocks < cap ? blocks : cap), 256, 0, st>>>(X, vals, meta, s, L, T, b, r,
                                                                      d_out, d_in, Y);
    count_launch(1);
    if (cudaGetLastError() != cudaSuccess) return SLIM_ERR_CUDA;
    // The decode kernels read this region as hand-over slots (all ones = empty): leave it as they expect it.
    if (r > 0 && cudaMemsetAsync(T, 0xFF, (size_t)b * r * sizeof(float), st) != cudaSuccess) return SLIM_ERR_CUDA;
    return SLIM_OK;
}

}  // namespace slim
