// slim_mask_top2: the 2:4 mask of the pipeline's second step (Sec. 3, Fig. 1; metric: Sec. 3.2, the product
// of weight and input magnitudes).  One thread per group of four along d_in: metric |code| * xbar[k] (one
// binary32 multiplication; xbar == nullptr: |code|), the two largest kept, equal metrics to the lower
// index.  HBM-bound: 1 B read + 1 B written per weight.
#include "common.cuh"

namespace slim {

__global__ void mask_top2_kernel(const int8_t* __restrict__ codes, const float* __restrict__ xbar, int d_in, size_t n_groups,
                                 uint8_t* __restrict__ mask, uint32_t* status)
{
    const size_t gi = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (gi >= n_groups) return;
    const int gpr = d_in / 4;                               // groups per row
    const int k0 = 4 * (int)(gi % (size_t)gpr);
    const char4 c = reinterpret_cast<const char4*>(codes)[gi];
    float m[4] = {fabsf((float)c.x), fabsf((float)c.y), fabsf((float)c.z), fabsf((float)c.w)};
    if (xbar) {
        const float4 x = *reinterpret_cast<const float4*>(xbar + k0);
        if (!(x.x >= 0.f && x.x <= 3.0e38f && x.y >= 0.f && x.y <= 3.0e38f && x.z >= 0.f && x.z <= 3.0e38f && x.w >= 0.f && x.w <= 3.0e38f))
            flag_error(status, SLIM_ERR_INVALID_ARG);
        m[0] = __fmul_rn(m[0], x.x); m[1] = __fmul_rn(m[1], x.y); m[2] = __fmul_rn(m[2], x.z); m[3] = __fmul_rn(m[3], x.w);
    }
    uint32_t out = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int beaten = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (j != i && (m[j] > m[i] || (m[j] == m[i] && j < i))) ++beaten;
        out |= (uint32_t)(beaten < 2) << (8 * i);
    }
    reinterpret_cast<uint32_t*>(mask)[gi] = out;
}

slim_status_t launch_mask_top2(const int8_t* codes, const float* xbar, int d_out, int d_in, uint8_t* mask, uint32_t* status_dev,
                               cudaStream_t st)
{
    const size_t n_groups = (size_t)d_out * (size_t)(d_in / 4);
    mask_top2_kernel<<<(unsigned)((n_groups + 255) / 256), 256, 0, st>>>(codes, xbar, d_in, n_groups, mask, status_dev);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

}  // namespace slim
