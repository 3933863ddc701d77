// Packer / metadata encoder and its inverse.  Integer-only, HBM-bound:
// 2 B read + 0.375 B written per dense weight.
#include "common.cuh"

namespace slim {

// One thread handles 16 consecutive columns (four groups) of one row: two
// 16-byte loads, one 4-byte and one 2-byte store.  Consecutive threads walk
// consecutive columns, so a warp reads 512 contiguous bytes of codes and mask.
__global__ void __launch_bounds__(256)
pack_kernel(const int8_t* __restrict__ codes, const uint8_t* __restrict__ mask,
            long long n_chunks, uint8_t* __restrict__ vals, uint8_t* __restrict__ meta,
            uint32_t* status_dev)
{
    uint32_t err = 0;
    for (long long c = blockIdx.x * (long long)blockDim.x + threadIdx.x; c < n_chunks;
         c += (long long)gridDim.x * blockDim.x) {
        const int4 cv = __ldg(reinterpret_cast<const int4*>(codes) + c);
        const int4 mv = __ldg(reinterpret_cast<const int4*>(mask) + c);
        const uint32_t cw[4] = {(uint32_t)cv.x, (uint32_t)cv.y, (uint32_t)cv.z, (uint32_t)cv.w};
        const uint32_t mw[4] = {(uint32_t)mv.x, (uint32_t)mv.y, (uint32_t)mv.z, (uint32_t)mv.w};
        uint32_t vout = 0, mout = 0;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            int pos[2] = {0, 0};
            int v[2] = {0, 0};
            int kept = 0;
            bool bad_code = false;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const bool k = ((mw[g] >> (8 * i)) & 0xFFu) != 0;
                if (k) {
                    const int code = (int)(int8_t)((cw[g] >> (8 * i)) & 0xFFu);
                    if (code < -8 || code > 7) bad_code = true;
                    if (kept < 2) { pos[kept] = i; v[kept] = code; }
                    ++kept;
                }
            }
            uint32_t vb, mb;
            if (kept > 2 || bad_code) {
                err |= 1u << (kept > 2 ? SLIM_ERR_BAD_MASK : SLIM_ERR_CODE_RANGE);
                vb = 0; mb = 0x4;
            } else {
                if (kept == 0) { pos[0] = 0; pos[1] = 1; }
                else if (kept == 1) {
                    // complete with the lowest position not kept, keep ascending order
                    if (pos[0] == 0) { pos[1] = 1; }
                    else { pos[1] = pos[0]; v[1] = v[0]; pos[0] = 0; v[0] = 0; }
                }
                vb = ((uint32_t)v[0] & 0xFu) | (((uint32_t)v[1] & 0xFu) << 4);
                mb = (uint32_t)pos[0] | ((uint32_t)pos[1] << 2);
            }
            vout |= vb << (8 * g);
            mout |= mb << (4 * g);
        }
        reinterpret_cast<uint32_t*>(vals)[c] = vout;
        reinterpret_cast<uint16_t*>(meta)[c] = (uint16_t)mout;
    }
    if (err && status_dev) atomicOr(status_dev, err);
}

__global__ void __launch_bounds__(256)
unpack_kernel(const uint8_t* __restrict__ vals, const uint8_t* __restrict__ meta,
              long long n_chunks, int8_t* __restrict__ codes, uint8_t* __restrict__ mask)
{
    for (long long c = blockIdx.x * (long long)blockDim.x + threadIdx.x; c < n_chunks;
         c += (long long)gridDim.x * blockDim.x) {
        const uint32_t vw = __ldg(reinterpret_cast<const uint32_t*>(vals) + c);
        const uint32_t mw = __ldg(reinterpret_cast<const uint16_t*>(meta) + c);
        uint32_t cw[4], kw[4];
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const uint32_t vb = (vw >> (8 * g)) & 0xFFu;
            const uint32_t m = (mw >> (4 * g)) & 0xFu;
            const int p0 = m & 3, p1 = (m >> 2) & 3;
            const int c0 = ((int)((vb & 0xFu) << 28)) >> 28;
            const int c1 = ((int)((vb >> 4) << 28)) >> 28;
            uint32_t cwv = ((uint32_t)c0 & 0xFFu) << (8 * p0);
            cwv = (cwv & ~(0xFFu << (8 * p1))) | (((uint32_t)c1 & 0xFFu) << (8 * p1));
            cw[g] = cwv;
            kw[g] = (1u << (8 * p0)) | (1u << (8 * p1));
        }
        reinterpret_cast<int4*>(codes)[c] = make_int4((int)cw[0], (int)cw[1], (int)cw[2], (int)cw[3]);
        if (mask) reinterpret_cast<int4*>(mask)[c] = make_int4((int)kw[0], (int)kw[1], (int)kw[2], (int)kw[3]);
    }
}

static int grid_for(long long n_chunks, int sm_count) {
    long long blocks = (n_chunks + 255) / 256;
    long long cap = (long long)sm_count * 8;     // grid-stride over a full machine
    return (int)(blocks < cap ? (blocks < 1 ? 1 : blocks) : cap);
}

slim_status_t launch_pack(const int8_t* codes, const uint8_t* mask, int d_out, int d_in,
                          uint8_t* vals, uint8_t* meta, uint32_t* status_dev, cudaStream_t st)
{
    slim_status_t err;
    const DeviceInfo* di = device_info(&err);
    if (!di) return err;
    const long long n_chunks = (long long)d_out * d_in / 16;
    pack_kernel<<<grid_for(n_chunks, di->sm_count), 256, 0, st>>>(codes, mask, n_chunks, vals, meta, status_dev);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

slim_status_t launch_unpack(const uint8_t* vals, const uint8_t* meta, int d_out, int d_in,
                            int8_t* codes, uint8_t* mask, cudaStream_t st)
{
    slim_status_t err;
    const DeviceInfo* di = device_info(&err);
    if (!di) return err;
    const long long n_chunks = (long long)d_out * d_in / 16;
    unpack_kernel<<<grid_for(n_chunks, di->sm_count), 256, 0, st>>>(vals, meta, n_chunks, codes, mask);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

}  // namespace slim
