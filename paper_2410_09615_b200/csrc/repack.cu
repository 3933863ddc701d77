// slim_repack_tiled: the decode-tiled copy of a packed weight (layout in include/slim.h).
// Bytes only move; one thread builds one 32-bit word of the output.
#include "common.cuh"

namespace slim {

__global__ void repack_tiled_kernel(const uint8_t* __restrict__ vals, const uint8_t* __restrict__ meta, int d_in, int nblk,
                                    int tiles, size_t n_words, uint32_t* __restrict__ out)
{
    const size_t wi = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (wi >= n_words) return;
    const int k = (int)(wi % 384);                       // word inside the 1536-byte piece
    // pieces are stored by groups of four tiles: in a group block after block, in a block the group's four
    // tiles; tiles past d_out / 16 are padding (stored zeros at positions 0 and 1)
    const size_t piece = wi / 384;
    const int rem = (int)(piece % (size_t)(4 * nblk));
    const int tile = 4 * (int)(piece / (size_t)(4 * nblk)) + (rem & 3), blk = rem >> 2;
    if (tile >= tiles) { out[wi] = k < 256 ? 0u : 0x44444444u; return; }
    const size_t vrow = (size_t)d_in / 4, mrow = (size_t)d_in / 8;
    uint32_t w = 0;
    if (k < 256) {
        // value word of step j, lane (g, t): four value bytes, nibbles 4 bits apart in each half-word
        const int j = 4 * (k >> 7) + (k & 3), lane = (k & 127) >> 2, g = lane >> 2, t = lane & 3;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = 16 * tile + g + 8 * (i & 1);
            const int group = 64 * blk + 8 * j + 4 * (i >> 1) + t;
            const uint32_t B = vals[(size_t)row * vrow + group];
            w |= (B & 0xFu) << (4 * i);
            w |= (B >> 4) << (16 + 4 * i);
        }
    } else {
        // index word of lane (g, t), step 4 (t / 2) + jj: 16 columns of row g and of row g + 8
        const int k2 = k - 256, lane = k2 >> 2, jj = k2 & 3, g = lane >> 2, t = lane & 3;
        const int j = 4 * (t >> 1) + jj;
        const uint8_t* m0 = meta + (size_t)(16 * tile + g) * mrow + 32 * blk + 4 * j + 2 * (t & 1);
        const uint8_t* m1 = m0 + 8 * mrow;
        w = (uint32_t)m0[0] | ((uint32_t)m0[1] << 8) | ((uint32_t)m1[0] << 16) | ((uint32_t)m1[1] << 24);
    }
    out[wi] = w;
}

slim_status_t launch_repack_tiled(const uint8_t* vals, const uint8_t* meta, int d_out, int d_in, uint8_t* out, cudaStream_t st)
{
    const size_t n_words = (size_t)((d_out + 63) / 64 * 64) * (size_t)d_in / 8 * 3 / 4;
    const unsigned blocks = (unsigned)((n_words + 255) / 256);
    repack_tiled_kernel<<<blocks, 256, 0, st>>>(vals, meta, d_in, d_in / 256, d_out / 16, n_words, reinterpret_cast<uint32_t*>(out));
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

}  // namespace slim
