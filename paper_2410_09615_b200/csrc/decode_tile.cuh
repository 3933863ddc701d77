// Warp-level building blocks of the decode kernel: shared-memory fragment reads,
// the int4 -> bf16 expansion and the two tensor-core steps (sparse weight block,
// dense adapter step).  Everything here works on data that is already in shared
// memory; the kernel file owns the pipeline around it.
#pragma once
#include "common.cuh"

namespace slim {
namespace dt {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Shared-memory reads by 32-bit shared address.  Plain loads, so that the compiler may move them
// ahead of the arithmetic of the previous block; the barrier waits and arrivals around a slot carry
// memory clobbers, which keeps the reads inside the slot's lifetime.
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    return *reinterpret_cast<const uint4*>(__cvta_shared_to_generic(addr));
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    return *reinterpret_cast<const uint32_t*>(__cvta_shared_to_generic(addr));
}

// Byte offset inside a TMA tile of 128-byte rows stored with the 128-byte swizzle (tile
// base aligned to 1024 bytes): the 16-byte chunk index is XOR-ed with the row number mod 8.
__device__ __forceinline__ uint32_t swz128(int row, int byte_off) {
    return (uint32_t)(row * 128 + ((((byte_off >> 4) ^ row) & 7) << 4) + (byte_off & 15));
}

// D(16x8, fp32) += A(16x32 bf16, 2:4 sparse, stored 16x16) * B(32x8 bf16).
// SEL picks which thread pair of every quad supplies the metadata word.
template <int SEL>
__device__ __forceinline__ void mma_sp_16832(float* c, const uint32_t* a, const uint4& b, uint32_t e) {
    asm(
        "mma.sp::ordered_metadata.sync.aligned.m16n8k32.row.col.f32.bf16.bf16.f32 "
        "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9,%10,%11}, {%0,%1,%2,%3}, %12, %13;"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w), "r"(e), "n"(SEL));
}
// D(16x8, fp32) += A(16x16 bf16) * B(16x8 bf16)
__device__ __forceinline__ void mma_16816(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
    asm(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 "
        "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Two int4 codes, the first in bits 0-3 and the second in bits 16-19 of `x` (other bits
// arbitrary), as an exact bf16x2: nibble ^ 8 in the mantissa of 128.0 is 128 + (v + 8);
// subtracting 136 leaves v in [-8, 7].
__device__ __forceinline__ uint32_t nibbles_to_bf16x2(uint32_t x) {
    uint32_t y;
    asm("lop3.b32 %0, %1, %2, %3, 0x6a;" : "=r"(y) : "r"(x), "r"(0x000F000Fu), "r"(0x43084308u));
    __nv_bfloat162 v = *reinterpret_cast<__nv_bfloat162*>(&y);
    const uint32_t bias_bits = 0x43084308u;   // 136.0 twice
    v = __hsub2(v, *reinterpret_cast<const __nv_bfloat162*>(&bias_bits));
    return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ uint32_t word_of(const uint4& v, int i) {
    return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w;
}

struct LaneCtx {
    int lane, g, t;           // lane, lane / 4, lane % 4
};
__device__ __forceinline__ LaneCtx make_lane_ctx(int lane) {
    LaneCtx c;
    c.lane = lane; c.g = lane >> 2; c.t = lane & 3;
    return c;
}

// Activations of one 256-column block as sparse B fragments: step j, n-tile h.
// Shared-memory layout of an activation (or T) slice, "fragment order":
//   [k-step of 32 columns][token < b][t = 0..3][i = 0..3]  32-bit words,
//   word = X[token][32 step + 2 t + 8 i .. + 1]
// so one thread's four B registers of a step are one 16-byte read, and the reads of
// a warp cover consecutive addresses.  Tokens >= b are not stored: their lanes use zeros.
template <int NT>
__device__ __forceinline__ void load_x_block(uint4 (&xf)[8][NT], uint32_t xs_addr, int step0, int b, const LaneCtx& lc) {
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int h = 0; h < NT; ++h) {
            const int tok = lc.g + 8 * h;
            xf[j][h] = tok < b ? lds128(xs_addr + (uint32_t)((((step0 + j) * b + tok) * 4 + lc.t) * 16)) : make_uint4(0, 0, 0, 0);
        }
}
template <int NT>
__device__ __forceinline__ void load_x_step(uint4 (&xb)[NT], uint32_t xs_addr, int step, int b, const LaneCtx& lc) {
#pragma unroll
    for (int h = 0; h < NT; ++h) {
        const int tok = lc.g + 8 * h;
        xb[h] = tok < b ? lds128(xs_addr + (uint32_t)(((step * b + tok) * 4 + lc.t) * 16)) : make_uint4(0, 0, 0, 0);
    }
}

// One 16-row x 256-column block of the decode-tiled weight (1536 bytes in shared memory,
// layout in include/slim.h) against the block's activations: eight steps of 32 columns.
// A value word holds the thread's four A-register pairs of one step, nibbles 4 bits apart in
// each half-word, so a register costs one shift, one logic operation and one bf16 subtraction;
// an index word is the step's metadata as the instruction takes it (lanes 2 SEL and 2 SEL + 1
// of a quad supply columns 0-15 and 16-31; bits 0-15 row g, bits 16-31 row g + 8): steps 0-3
// use SEL 0, steps 4-7 SEL 1, so every lane holds the words of four steps.
template <int NT>
__device__ __forceinline__ void sparse_block(float (&acc)[NT][4], uint32_t blk_addr, const uint4 (&xf)[8][NT], const LaneCtx& lc) {
    const uint4 va = lds128(blk_addr + lc.lane * 16);
    const uint4 vb = lds128(blk_addr + 512 + lc.lane * 16);
    const uint4 me = lds128(blk_addr + 1024 + lc.lane * 16);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t w = word_of(j < 4 ? va : vb, j & 3);
        uint32_t a[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = nibbles_to_bf16x2(w >> (4 * i));
        const uint32_t e = word_of(me, j & 3);
#pragma unroll
        for (int h = 0; h < NT; ++h) {
            if (j < 4) mma_sp_16832<0>(acc[h], a, xf[j][h], e);
            else       mma_sp_16832<1>(acc[h], a, xf[j][h], e);
        }
    }
}

// One step of 32 columns of a dense bf16 tile (16 rows x 64 columns = 128-byte rows,
// 128-byte swizzle, tile base a multiple of 2048 bytes inside a 1024-byte aligned box; `half` = which 32 columns) against B fragments in fragment order:
// two m16n8k16 MMAs in natural column order.
template <int NT>
__device__ __forceinline__ void dense_step(float (&acc)[NT][4], uint32_t tile_addr, int half, const uint4 (&xb)[NT], const LaneCtx& lc) {
    uint32_t a0[4], a1[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        a0[i] = lds32(tile_addr + swz128(lc.g, 64 * half + 16 * i + 4 * lc.t));
        a1[i] = lds32(tile_addr + swz128(lc.g + 8, 64 * half + 16 * i + 4 * lc.t));
    }
#pragma unroll
    for (int h = 0; h < NT; ++h) {
        mma_16816(acc[h], a0[0], a1[0], a0[1], a1[1], xb[h].x, xb[h].y);
        mma_16816(acc[h], a0[2], a1[2], a0[3], a1[3], xb[h].z, xb[h].w);
    }
}

}  // namespace dt
}  // namespace slim
