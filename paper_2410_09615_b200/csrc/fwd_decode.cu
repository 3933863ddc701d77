// Decode-phase forward (b <= 16): one persistent cooperative kernel that
// streams the packed weight and the adapters from HBM exactly once.
//
// Tensor-core mapping.  The batch is the N dimension of warp-level MMAs (one or
// two n-tiles of 8 tokens), so the kernel stays bandwidth-bound up to b = 16:
//   * packed weight rows are the SPARSE A operand of
//     mma.sp::ordered_metadata.m16n8k32 (bf16 x bf16 -> fp32): the value byte of
//     one 2:4 group is exactly one thread's A-register pair and a 32-bit word of
//     the index array is the instruction's metadata for one row, so decoding is
//     nibble -> exact bf16 integer and nothing else;
//   * adapter rows (R, then L) are the dense A operand of mma.m16n8k16; inside a
//     32-column block the k order is permuted so that a thread's A and B
//     fragments are single 16-byte reads.
//
// Data movement.  Every operand travels global -> shared memory as TMA tiles
// (cp.async.bulk.tensor.2d, 128-byte rows, 128-byte swizzle, mbarrier
// completion): the CTA's slice of the activations once, then a ring of 16 KB
// slots for the streamed matrices.  The lanes of a ninth, producer warp issue
// the tiles of a chunk in parallel (a thread is held about 160 cycles by every
// tile request it starts); the eight consumer warps read MMA fragments from shared memory.
//
// Work split.  d_in is cut into 256-column blocks and into k-slices of <= 8
// blocks; a CTA belongs to one slice, one block per consumer warp.  Each CTA
// first takes its share of R chunks (16 rows x 512 columns), then its share of
// 16-row weight tiles; both leave split-K partial tiles (fp32, MMA fragment
// order) in the workspace.  A tenth, service warp of one CTA per 16 columns of
// T = X R^T sums that piece's partials and publishes it in bf16 while the
// weight stream is still running.  Finally every CTA finishes 16-row output
// tiles:  Y = s * sum(partials) + T L^T, with the L rows already prefetched
// into the ring.
//
// Cross-CTA hand-over without fences.  A partial-sum slot is written once and
// read by exactly one thread: it holds a reserved NaN pattern while empty, the
// reader polls the slot itself until the pattern is gone and puts the pattern
// back for the next call.  The bf16 pieces of T have many readers, so each
// 8-byte entry carries the number of the call that wrote it; the call number
// comes from a counter every CTA increments when it leaves.  All polls are
// bounded; an expired one sets SLIM_ERR_TIMEOUT and the kernel runs on to its
// end (the launch is cooperative, so all CTAs are resident).  Reductions have a
// fixed order: results are bit-identical from run to run.
#include <cuda.h>
#include "common.cuh"

namespace slim {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kProducerWarp = kConsumerWarps;
constexpr int kServiceWarp = kConsumerWarps + 1;
constexpr int kServiceWarps = 2;
constexpr int kDecodeThreads = kConsumerThreads + 32 + 32 * kServiceWarps;
constexpr int kMaxDecodeRank = 3072;
constexpr int kMaxSlices = 16;
constexpr int kMaxSlots = 16;
constexpr uint32_t kPollLimit = 1u << 22;                  // polls of a global slot
constexpr uint32_t kMbarSpinLimit = 1u << 26;              // shared-memory barriers
constexpr int kRChunkCols = 512;                           // columns of one R chunk
constexpr int kLChunkCols = 512;                           // columns (of r) of one L chunk
constexpr int kSubTile = 2048;                             // one TMA box: 16 rows x 128 bytes
constexpr int kSlotBytes = 8 * kSubTile;
constexpr size_t kSmemBudget = 227 * 1024;
// The published T sits at a fixed place in the workspace (right after the call counter) so
// that calls of different shapes sharing a workspace never read one kind of slot as the other.
constexpr size_t kTfinalBytes = kDecodeTfinalBytes;
static_assert(16 * (size_t)(((kMaxDecodeRank + 63) / 64 * 64 + 32) / 2) * 8 <= kTfinalBytes, "published T does not fit its region");
constexpr uint32_t kEmpty = 0xFFFFFFFFu;                   // "no value yet" in a partial-sum slot
constexpr uint32_t kNanBits = 0x7FFFFFFFu;                 // what a computed all-ones NaN is stored as

struct DecodeParams {
    const __nv_bfloat16* X; const uint8_t* vals; const uint8_t* meta;
    const __nv_bfloat16* L; const __nv_bfloat16* R; __nv_bfloat16* Y;
    const __nv_bfloat16* Ls; const __nv_bfloat16* Rs;     // quantized adapters: scales [d_out][ceil(r/128)], [r][d_in/128]
    uint32_t* Ppart;              // [KS][tilesW][frag]      fp32 bits or kEmpty
    uint32_t* Tpart;              // [tilesR][QT][frag]      fp32 bits or kEmpty
    uint2* Tfinal;                // [NT*8][r_pad/2]         {bf16 pair, call number}
    unsigned long long* departures;   // CTAs that ever left a call on this workspace
    uint32_t* status;
    float s;
    int b, r, d_out, d_in;
    int KS, nblk, G, QT, r_pad;
    int chunk_blocks;             // 256-column blocks of one R chunk: 2 (bf16 adapters), 8 (quantized adapters)
    int l_direct;                 // quantized adapters whose rows of L codes are no 16-byte multiples: read with plain loads
    const uint8_t* Lq;            // codes of L (used when l_direct)
    int n_slots;
};

// Optional timeline: built with -DSLIM_DECODE_TRACE, thread 0 of every CTA records
// the global timer at the phase boundaries (read back with slim_debug_read_trace).
#ifdef SLIM_DECODE_TRACE
__device__ unsigned long long g_trace[256 * 32];
#define STAMP(i) do { if (threadIdx.x == 0) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); g_trace[blockIdx.x * 32 + (i)] = t_; } } while (0)
#else
#define STAMP(i) do { } while (0)
#endif

// ------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Bounded wait for the phase with the given parity; returns false on expiry.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_u32(bar);
    for (uint32_t it = 0; it < kMbarSpinLimit; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}
// Has the phase completed?  Does not wait: the answer takes a couple of hundred cycles to come back, so it
// is asked one slot ahead and looked at when the slot is needed.
__device__ __forceinline__ uint32_t mbar_test(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return done;
}
// One TMA tile (box of the tensor behind `tmap`, starting at element column x,
// row y) into shared memory; completion in bytes on `bar`.
__device__ __forceinline__ void tma_tile(void* dst, const CUtensorMap* tmap, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 :: "r"(smem_u32(dst)), "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
// Byte address inside a 128-byte-swizzled tile: the 16-byte chunk index is
// XOR-ed with the row number modulo 8.
__device__ __forceinline__ uint32_t swz(int row, int byte_off) {
    return (uint32_t)(row * 128 + ((((byte_off >> 4) ^ row) & 7) << 4) + (byte_off & 15));
}
__device__ __forceinline__ void consumer_sync() {          // the eight consumer warps only
    asm volatile("bar.sync 1, %0;" :: "n"(kConsumerThreads) : "memory");
}
__device__ __forceinline__ uint4 lds128(const void* p) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(smem_u32(p)));
    return v;
}
__device__ __forceinline__ uint32_t lds32(const void* p) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)));
    return v;
}
// Device-scope accesses that bypass L1: the hand-over slots.
__device__ __forceinline__ uint32_t ld_gpu(const uint32_t* p) {
    uint32_t v;
#ifdef SLIM_LD_VOLATILE
    asm volatile("ld.volatile.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
#else
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
#endif
    return v;
}
// A published entry of T is read and written as ONE 64-bit access: only a scalar access is
// guaranteed to be seen whole (value and call number together).
__device__ __forceinline__ uint2 ld_gpu2(const uint2* p) {
    unsigned long long u;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(u) : "l"(p) : "memory");
    return make_uint2((uint32_t)u, (uint32_t)(u >> 32));
}
__device__ __forceinline__ void st_gpu(uint32_t* p, uint32_t v) {
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void st_gpu2(uint2* p, uint2 v) {
    const unsigned long long u = ((unsigned long long)v.y << 32) | v.x;
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" :: "l"(p), "l"(u) : "memory");
}
__device__ __forceinline__ unsigned long long ld_gpu64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t slot_bits(float v) {    // fp32 bits that never equal kEmpty
    const uint32_t u = __float_as_uint(v);
    return u == kEmpty ? kNanBits : u;
}

// D(16x8, fp32) += A(16x32 bf16, 2:4 sparse, stored 16x16) * B(32x8 bf16).
// SEL picks which thread pair of every quad supplies the metadata word.
template <int SEL>
__device__ __forceinline__ void mma_sp_16832(float* c, const uint32_t* a, const uint32_t* bfrag, uint32_t e) {
    asm volatile(
        "mma.sp::ordered_metadata.sync.aligned.m16n8k32.row.col.f32.bf16.bf16.f32 "
        "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9,%10,%11}, {%0,%1,%2,%3}, %12, %13;"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]),
          "r"(bfrag[0]), "r"(bfrag[1]), "r"(bfrag[2]), "r"(bfrag[3]), "r"(e), "n"(SEL));
}
// D(16x8, fp32) += A(16x16 bf16) * B(16x8 bf16)
__device__ __forceinline__ void mma_16816(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 "
        "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Byte `t` of `w` holds one 2:4 group (two int4 codes).  Returns the two codes
// as an exact bf16x2: nibble ^ 8 in the mantissa of 128.0 gives 128 + (v + 8);
// subtracting 136 leaves v in [-8, 7].
__device__ __forceinline__ uint32_t decode_group(uint32_t w, uint32_t byte_sel) {
    uint32_t x;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(x) : "r"(w), "r"(w >> 4), "r"(byte_sel));
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

// Quantized adapters.  Two int4 codes at bits 0-3 and 16-19 of `x` (other bits arbitrary) as an exact bf16x2.
__device__ __forceinline__ uint32_t nib_pair(uint32_t x) {
    uint32_t y;
    asm("lop3.b32 %0, %1, %2, %3, 0x6a;" : "=r"(y) : "r"(x), "r"(0x000F000Fu), "r"(0x43084308u));
    __nv_bfloat162 v = *reinterpret_cast<__nv_bfloat162*>(&y);
    const uint32_t bias_bits = 0x43084308u;
    v = __hsub2(v, *reinterpret_cast<const __nv_bfloat162*>(&bias_bits));
    return *reinterpret_cast<uint32_t*>(&v);
}
// A word of eight codes c0..c7 (two per byte, even column low) gives, shifted by 4 i, the pair (c_i, c_{i+4}):
// the dense operand of a quantized adapter pairs columns four apart, and the other operand's eight
// consecutive bf16 values (c0 c1 | c2 c3 | c4 c5 | c6 c7) are put in the same order.
__device__ __forceinline__ uint4 pair_four_apart(const uint4& v) {
    uint4 o;
    asm("prmt.b32 %0, %1, %2, 0x5410;" : "=r"(o.x) : "r"(v.x), "r"(v.z));
    asm("prmt.b32 %0, %1, %2, 0x7632;" : "=r"(o.y) : "r"(v.x), "r"(v.z));
    asm("prmt.b32 %0, %1, %2, 0x5410;" : "=r"(o.z) : "r"(v.y), "r"(v.w));
    asm("prmt.b32 %0, %1, %2, 0x7632;" : "=r"(o.w) : "r"(v.y), "r"(v.w));
    return o;
}

// ------------------------------------------------------------ work split
// Computed identically by every warp role.
struct Share {
    int ks, grp;             // k-slice and position inside the slice's CTA group (-1: no streaming work)
    int blk_begin, nb;       // 256-column blocks of the slice
    int Qk;                  // R chunks per 16-row R tile in this slice
    int qoff;                // index of the slice's first chunk among a tile's QT partial slots
    int r_begin, r_count;    // R chunk units [r_begin, r_begin + r_count)
    int w_begin, w_count;    // weight tiles
};

__device__ __forceinline__ Share make_share(const DecodeParams& p, int cta) {
    Share sh;
    const int tilesW = p.d_out / 16, tilesR = p.r / 16;
    if (cta >= p.KS * p.G) {
        sh.ks = 0; sh.grp = -1; sh.blk_begin = 0; sh.nb = 0; sh.Qk = 0; sh.qoff = 0;
        sh.r_begin = sh.r_count = sh.w_begin = sh.w_count = 0;
        return sh;
    }
    sh.ks = cta % p.KS; sh.grp = cta / p.KS;
    sh.blk_begin = (int)((long long)sh.ks * p.nblk / p.KS);
    sh.nb = (int)((long long)(sh.ks + 1) * p.nblk / p.KS) - sh.blk_begin;
    sh.Qk = (sh.nb + p.chunk_blocks - 1) / p.chunk_blocks;
    int qoff = 0;
    for (int k = 0; k < sh.ks; ++k) {
        const int nbk = (int)((long long)(k + 1) * p.nblk / p.KS) - (int)((long long)k * p.nblk / p.KS);
        qoff += (nbk + p.chunk_blocks - 1) / p.chunk_blocks;
    }
    sh.qoff = qoff;
    // R chunks: the first CTAs of the group take the remainder; weight tiles: the last ones do
    const int UR = tilesR * sh.Qk, G = p.G;
    sh.r_count = UR / G + (sh.grp < UR % G ? 1 : 0);
    sh.r_begin = sh.grp * (UR / G) + (sh.grp < UR % G ? sh.grp : UR % G);
    const int rem = tilesW % G;
    sh.w_count = tilesW / G + (sh.grp >= G - rem ? 1 : 0);
    sh.w_begin = sh.grp * (tilesW / G) + (sh.grp > G - rem ? sh.grp - (G - rem) : 0);
    return sh;
}

// Sum the consumer warps' partial tiles (fragment order) through shared memory.
// Cross-warp sums go through a ring of buffers in shared memory: a buffer is written again only
// two consumer barriers after it was read (the weight phase uses two buffers per barrier).
constexpr int kRedBufs = 4;

template <int NT>
__device__ __forceinline__ float block_tile_sum(float* red, const float (&acc)[NT][4], bool active, int n_active) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int frag = NT * 128;
    if (active) {
#pragma unroll
        for (int h = 0; h < NT; ++h)
#pragma unroll
            for (int q = 0; q < 4; ++q) red[warp * frag + (h * 4 + q) * 32 + lane] = acc[h][q];
    }
    consumer_sync();
    float sum = 0.f;
    if (threadIdx.x < frag)
        for (int w = 0; w < n_active; ++w) sum += red[w * frag + threadIdx.x];
    return sum;
}

// The same for two tiles with one barrier: a barrier and its skew cost as much as a tile's MMAs.
template <int NT>
__device__ __forceinline__ float2 block_tile_sum2(float* red0, float* red1, const float (&acc0)[NT][4],
                                                  const float (&acc1)[NT][4], bool active, int n_active) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int frag = NT * 128;
    if (active) {
#pragma unroll
        for (int h = 0; h < NT; ++h)
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                red0[warp * frag + (h * 4 + q) * 32 + lane] = acc0[h][q];
                red1[warp * frag + (h * 4 + q) * 32 + lane] = acc1[h][q];
            }
    }
    consumer_sync();
    float2 sum = make_float2(0.f, 0.f);
    if (threadIdx.x < frag)
        for (int w = 0; w < n_active; ++w) { sum.x += red0[w * frag + threadIdx.x]; sum.y += red1[w * frag + threadIdx.x]; }
    return sum;
}

// Partial-sum slots, `n` (<= kMaxSlices) of them `stride` words apart.
// slots_request reads them all once; slots_finish re-reads together those still
// empty until every one holds a value, adds the values in slot order and marks
// the slots empty again.
struct SlotBatch { uint32_t v[kMaxSlices]; };

__device__ __forceinline__ void slots_request(SlotBatch& sb, const uint32_t* first, size_t stride, int n) {
#pragma unroll
    for (int i = 0; i < kMaxSlices; ++i) sb.v[i] = i < n ? ld_gpu(first + (size_t)i * stride) : 0u;
}

__device__ __forceinline__ float slots_finish(SlotBatch& sb, uint32_t* first, size_t stride, int n, bool* ok) {
    for (uint32_t spins = 0;; ++spins) {
        bool all = true;
#pragma unroll
        for (int i = 0; i < kMaxSlices; ++i) all = all && sb.v[i] != kEmpty;
        if (all) break;
        if (spins > kPollLimit) { *ok = false; break; }
#pragma unroll
        for (int i = 0; i < kMaxSlices; ++i)
            if (sb.v[i] == kEmpty) sb.v[i] = ld_gpu(first + (size_t)i * stride);
    }
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < kMaxSlices; ++i) {
        if (i < n) {
            sum += __uint_as_float(sb.v[i]);
            st_gpu(first + (size_t)i * stride, kEmpty);
        }
    }
    return sum;
}

__device__ __forceinline__ float take_slots(uint32_t* first, size_t stride, int n, bool* ok) {
    SlotBatch sb;
    slots_request(sb, first, stride, n);
    return slots_finish(sb, first, stride, n, ok);
}

// QA: the adapters are quantized (int4 codes with one bf16 scale per 128 elements of a row, layout in
// include/slim.h): tmR / tmL then describe the code bytes, a chunk of 512 columns is two tiles of 256
// codes, a warp's 64 columns lie inside one group, so the warp multiplies exact integer codes and
// scales its accumulator rows once per chunk.
template <int NT, bool QA = false>
__global__ void __launch_bounds__(kDecodeThreads, 1)
decode_kernel(const DecodeParams p, const __grid_constant__ CUtensorMap tmX,
              const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmM,
              const __grid_constant__ CUtensorMap tmR, const __grid_constant__ CUtensorMap tmL)
{
    constexpr int frag = NT * 128;
    constexpr int x_sub = NT * 8 * 128;                    // one 64-column tile of the activations
    extern __shared__ unsigned char smem_raw[];
    // layout (1024-byte aligned for the swizzle): ring slots | X slice | Ts | red x2 | barriers
    unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char* xs = ring + (size_t)p.n_slots * kSlotBytes;
    __nv_bfloat16* Ts = reinterpret_cast<__nv_bfloat16*>(xs + 32 * x_sub);
    float* red_base = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(Ts) + (size_t)NT * 8 * p.r_pad * 2);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(red_base + kRedBufs * kConsumerWarps * frag);
    uint64_t* empty_bar = full_bar + kMaxSlots;
    uint64_t* x_bar = empty_bar + kMaxSlots;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int tilesW = p.d_out / 16, tilesR = p.r / 16;
    const int n_ctas = gridDim.x;
    const Share sh = make_share(p, blockIdx.x);
    const int n_slots = p.n_slots;
    // Chunks of quantized adapters are wider, so that a synchronisation covers more columns.  R: 2048 columns
    // of codes fill a ring slot, a warp owns a whole 256-column block (four sub-steps of 64 columns, two groups
    // of 128 with their own scales).  L: 1024 columns of r, a warp owns one group of 128 (two sub-steps), so
    // that all warps work on the ranks in use (r <= 1024 is one chunk per output tile).
    constexpr int kRC = QA ? 2048 : kRChunkCols, kLC = QA ? 1024 : kLChunkCols;
    const int l_chunks = p.r > 0 ? ceil_div(p.r, kLC) : 0;

    if (threadIdx.x == 0) {
        for (int i = 0; i < n_slots; ++i) { mbar_init(&full_bar[i], 1); mbar_init(&empty_bar[i], kConsumerWarps); }
        mbar_init(x_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    STAMP(0);
    if (warp == kProducerWarp) {
        // ============================ producer warp ============================
        uint32_t it = 0;
        bool ok = true;
        // Returns the slot once it is free; lane 0 arms its full barrier.  The whole warp waits:
        // a single waiting lane followed by a warp barrier costs some hundred nanoseconds per
        // tile.  (A tile may land before lane 0 has armed the barrier; the phase cannot
        // complete before that arrival.)
        int slot_i = 0;
        uint32_t phase = 0;
        auto acquire = [&](uint32_t bytes) -> int {
            const int slot = slot_i;
            if (it >= (uint32_t)n_slots) ok = mbar_wait(&empty_bar[slot], phase ^ 1) && ok;
            if (lane == 0) mbar_arrive_expect_tx(&full_bar[slot], bytes);
            ++it;
            if (++slot_i == n_slots) { slot_i = 0; phase ^= 1; }
            return slot;
        };
        // ---- R chunks: 16 rows x (256 or 512) columns of bf16 = 4 or 8 tiles of 64 columns
        for (int u = sh.r_begin; u < sh.r_begin + sh.r_count; ++u) {
            const int tile = u / sh.Qk, q = u % sh.Qk;
            const int cols = min(kRC, sh.nb * 256 - q * kRC);
            const int n_sub = QA ? cols / 256 : cols / 64;
            const int slot = acquire((uint32_t)n_sub * kSubTile);
            if (lane < n_sub) {
                const int x = QA ? (sh.blk_begin * 256 + q * kRC) / 2 + 128 * lane      // bytes of codes
                                 : sh.blk_begin * 256 + q * kRC + 64 * lane;
                tma_tile(ring + (size_t)slot * kSlotBytes + lane * kSubTile, &tmR, x, tile * 16, &full_bar[slot]);
            }
        }
        // ---- weight tiles: value bytes (128 per tile row = 2 blocks), then index bytes (4 blocks)
        const int v_sub = (sh.nb + 1) / 2, m_sub = (sh.nb + 3) / 4;
        for (int tile = sh.w_begin; tile < sh.w_begin + sh.w_count; ++tile) {
            const int slot = acquire((uint32_t)(v_sub + m_sub) * kSubTile);
            unsigned char* dst = ring + (size_t)slot * kSlotBytes;
            if (lane < v_sub)
                tma_tile(dst + lane * kSubTile, &tmV, sh.blk_begin * 64 + 128 * lane, tile * 16, &full_bar[slot]);
            else if (lane >= 4 && lane < 4 + m_sub)
                tma_tile(dst + lane * kSubTile, &tmM, sh.blk_begin * 32 + 128 * (lane - 4), tile * 16, &full_bar[slot]);
        }
        // ---- L chunks of the output tiles this CTA finishes (512 columns of r = 8 tiles)
        for (int tile = blockIdx.x; tile < tilesW && p.r > 0 && !(QA && p.l_direct); tile += n_ctas) {
            for (int lc = 0; lc < l_chunks; ++lc) {
                const int cols = min(kLC, p.r - lc * kLC);
                const int n_sub = QA ? ceil_div(cols, 256) : ceil_div(cols, 64);
                const int slot = acquire((uint32_t)n_sub * kSubTile);
                if (lane < n_sub)
                    tma_tile(ring + (size_t)slot * kSlotBytes + lane * kSubTile, &tmL,
                             QA ? lc * (kLC / 2) + 128 * lane : lc * kLC + 64 * lane, tile * 16, &full_bar[slot]);
            }
        }
        if (lane == 0 && !ok) flag_error(p.status, SLIM_ERR_TIMEOUT);
        return;      // the consumers wait for every tile this warp requested before they leave
    }

    if (warp >= kServiceWarp) {
        // ============================ service warps ============================
        // Sums the split-K partials of the 16-column pieces jt = c, c + n_ctas, ... of T,
        // rounds to bf16 and publishes {two neighbouring columns, call number}.
        if (p.r == 0 || (int)blockIdx.x >= tilesR) return;
        const uint32_t call = (uint32_t)(ld_gpu64(p.departures) / (unsigned)n_ctas) + 1u;
        bool ok = true;
        for (int jt = blockIdx.x; jt < tilesR; jt += n_ctas) {
            uint32_t* base = p.Tpart + (size_t)jt * p.QT * frag;
            // Fragment element f = (h*4 + q)*32 + ln is T[token 8h + 2(ln%4) + (q&1)][16 jt + ln/4 + 8(q>>1)]:
            // elements with ln/4 = 2i and 2i+1 (same h, q, ln%4) are neighbours along the column index.
            for (int e = (int)threadIdx.x - kServiceWarp * 32; e < frag / 2; e += 32 * kServiceWarps) {
                const int i = e & 3, t4 = (e >> 2) & 3, hq = e >> 4;
                const int f0 = hq * 32 + 8 * i + t4, f1 = f0 + 4;
                float s0 = 0.f, s1 = 0.f;
                for (int sl0 = 0; sl0 < p.QT; sl0 += kMaxSlices) {
                    const int n = min(kMaxSlices, p.QT - sl0);
                    s0 += take_slots(base + (size_t)sl0 * frag + f0, frag, n, &ok);
                    s1 += take_slots(base + (size_t)sl0 * frag + f1, frag, n, &ok);
                }
                const int h = hq >> 2, q = hq & 3;
                const int m = 8 * h + 2 * t4 + (q & 1);
                const int j = jt * 16 + 2 * i + 8 * (q >> 1);
                __nv_bfloat162 pr = __floats2bfloat162_rn(s0, s1);
                st_gpu2(p.Tfinal + (size_t)m * (p.r_pad / 2) + (j >> 1), make_uint2(*reinterpret_cast<uint32_t*>(&pr), call));
            }
        }
#ifdef SLIM_DECODE_TRACE
        if (lane == 0) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); g_trace[blockIdx.x * 32 + 20] = t_; }
#endif
        if (!ok && lane == 0) flag_error(p.status, SLIM_ERR_TIMEOUT);
        return;
    }

    // ================================ consumer warps ================================
    uint32_t it = 0;
    int red_buf = 0;
    bool ok = true;
    // Ring position kept as running (slot, phase); the next slot's barrier is asked about while the current
    // slot is being consumed (an answer takes about 200 cycles even when the phase is long complete).
    int c_slot = 0;
    uint32_t c_phase = 0, ahead = 0;                       // ahead: the current slot was already seen full
    auto wait_full = [&]() -> unsigned char* {
        if (!ahead) ok = mbar_wait(&full_bar[c_slot], c_phase) && ok;
        const int ns = c_slot + 1 == n_slots ? 0 : c_slot + 1;
        ahead = mbar_test(&full_bar[ns], ns == 0 ? c_phase ^ 1u : c_phase);
        return ring + (size_t)c_slot * kSlotBytes;
    };
    auto release = [&]() {
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[c_slot]);
        ++it;
        if (++c_slot == n_slots) { c_slot = 0; c_phase ^= 1u; }
    };
    auto next_red = [&]() -> float* {
        float* r = red_base + red_buf * kConsumerWarps * frag;
        red_buf = (red_buf + 1) & (kRedBufs - 1);
        return r;
    };
    // the number of this call on this workspace (read before any CTA of the call can have left)
    uint32_t call = 0;
    if (p.r > 0) call = (uint32_t)(ld_gpu64(p.departures) / (unsigned)n_ctas) + 1u;

    // The CTA's slice of the activations: 4 tiles of 64 columns per block, rows >= b read as zero.
    // Consumer warp 0 requests it (a warp's first tile request takes most of a microsecond; the
    // producer warp spends that time on the first R chunk instead).
    if (warp == 0 && sh.grp >= 0) {
        if (lane == 0) mbar_arrive_expect_tx(x_bar, (uint32_t)(sh.nb * 4 * x_sub));
        if (lane < sh.nb * 4) tma_tile(xs + lane * x_sub, &tmX, sh.blk_begin * 256 + 64 * lane, 0, x_bar);
    }
    if (sh.grp >= 0) ok = mbar_wait(x_bar, 0) && ok;       // the activation slice is in shared memory
    STAMP(1);

    // ---------------------------------------------------------------- phase R
    if (sh.r_count > 0) {
        // activations as dense B fragments: chunk q, sub-block jj (32 columns), n-tile h:
        // 16 bytes X[g + 8h][slice + 512 q + 64 warp + 32 jj + 8 t .. +8)
        uint4 xd[4][2][NT];
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
            for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                for (int h = 0; h < NT; ++h) {
                    const int tile64 = QA ? warp * 4 + q : q * 8 + warp;   // 64-column tile of the slice (quantized: q = sub-step of the warp's block)
                    xd[q][jj][h] = tile64 < sh.nb * 4 ? lds128(xs + tile64 * x_sub + swz(g + 8 * h, jj * 64 + t * 16))
                                                      : make_uint4(0, 0, 0, 0);
                    if (QA) xd[q][jj][h] = pair_four_apart(xd[q][jj][h]);
                }
        for (int u = sh.r_begin; u < sh.r_begin + sh.r_count; ++u) {
            const int tile = u / sh.Qk, q = u % sh.Qk;
            const int cols = min(kRC, sh.nb * 256 - q * kRC);
            const bool active = QA ? warp * 256 < cols : warp * 64 < cols;
            float scA0 = 1.f, scA1 = 1.f, scB0 = 1.f, scB1 = 1.f;   // quantized R: scales of rows g, g + 8 in the block's two groups
            if (QA && active) {
                const size_t grp = (size_t)((sh.blk_begin * 256 + q * kRC + warp * 256) >> 7), per_row = (size_t)(p.d_in >> 7);
                const __nv_bfloat16* s0 = p.Rs + (size_t)(tile * 16 + g) * per_row + grp;
                const __nv_bfloat16* s1 = p.Rs + (size_t)(tile * 16 + g + 8) * per_row + grp;
                scA0 = __bfloat162float(s0[0]); scB0 = __bfloat162float(s0[1]);
                scA1 = __bfloat162float(s1[0]); scB1 = __bfloat162float(s1[1]);
            }
            const unsigned char* base = wait_full();
            if (u == sh.r_begin) STAMP(2);
            float acc[NT][4];
#pragma unroll
            for (int h = 0; h < NT; ++h)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[h][e] = 0.f;
            if (QA && active) {
                // warp w owns block w of the chunk = tile w of 256 codes per row; sub-steps of 64 columns
                const unsigned char* sub = base + warp * kSubTile;
#pragma unroll
                for (int half = 0; half < 2; ++half) {             // the block's two groups of 128 columns
                    float part[NT][4];
#pragma unroll
                    for (int h = 0; h < NT; ++h)
#pragma unroll
                        for (int e = 0; e < 4; ++e) part[h][e] = 0.f;
#pragma unroll
                    for (int ss = 0; ss < 2; ++ss) {
                        const int sq = half * 2 + ss;
#pragma unroll
                        for (int jj = 0; jj < 2; ++jj) {
                            const uint32_t wa = lds32(sub + swz(g, sq * 32 + jj * 16 + t * 4));
                            const uint32_t wb = lds32(sub + swz(g + 8, sq * 32 + jj * 16 + t * 4));
                            uint32_t a[4], c[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) { a[i] = nib_pair(wa >> (4 * i)); c[i] = nib_pair(wb >> (4 * i)); }
#pragma unroll
                            for (int h = 0; h < NT; ++h) {
                                const uint4 xb = xd[sq][jj][h];
                                mma_16816(part[h], a[0], c[0], a[1], c[1], xb.x, xb.y);
                                mma_16816(part[h], a[2], c[2], a[3], c[3], xb.z, xb.w);
                            }
                        }
                    }
                    const float r0 = half ? scB0 : scA0, r1 = half ? scB1 : scA1;
#pragma unroll
                    for (int h = 0; h < NT; ++h) {
                        acc[h][0] = fmaf(part[h][0], r0, acc[h][0]); acc[h][1] = fmaf(part[h][1], r0, acc[h][1]);
                        acc[h][2] = fmaf(part[h][2], r1, acc[h][2]); acc[h][3] = fmaf(part[h][3], r1, acc[h][3]);
                    }
                }
            } else if (active) {
                // warp w owns the 64-column tile w of the chunk
                const unsigned char* sub = base + warp * kSubTile;
                uint4 ra[2], rb[2];
#pragma unroll
                for (int jj = 0; jj < 2; ++jj) {
                    ra[jj] = lds128(sub + swz(g, jj * 64 + t * 16));
                    rb[jj] = lds128(sub + swz(g + 8, jj * 64 + t * 16));
                }
#pragma unroll
                for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                    for (int h = 0; h < NT; ++h) {
                        // the chunk index is not a compile-time constant: select the fragment set
                        uint4 xb = xd[0][jj][h];
                        if (q == 1) xb = xd[1][jj][h];
                        if (q == 2) xb = xd[2][jj][h];
                        if (q == 3) xb = xd[3][jj][h];
                        mma_16816(acc[h], ra[jj].x, rb[jj].x, ra[jj].y, rb[jj].y, xb.x, xb.y);
                        mma_16816(acc[h], ra[jj].z, rb[jj].z, ra[jj].w, rb[jj].w, xb.z, xb.w);
                    }
            }
            release();
            const float sum = block_tile_sum<NT>(next_red(), acc, active, QA ? cols / 256 : min(kConsumerWarps, cols / 64));
            if (threadIdx.x < frag)
                st_gpu(p.Tpart + ((size_t)tile * p.QT + sh.qoff + q) * frag + threadIdx.x, slot_bits(sum));
        }
    }

    STAMP(3);
    // ---------------------------------------------------------------- phase W
    if (sh.w_count > 0) {
        // activations as sparse B fragments: step j, n-tile h, register i holds
        // X[g + 8h][slice + 256 warp + 32 j + 2 t + 8 i .. +1]
        const bool w_active = warp < sh.nb;
        uint32_t xf[8][NT][4];
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int h = 0; h < NT; ++h)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int col = 32 * j + 2 * t + 8 * i;          // inside the warp's 256-column block
                    xf[j][h][i] = w_active ? lds32(xs + (warp * 4 + (col >> 6)) * x_sub + swz(g + 8 * h, (col & 63) * 2)) : 0u;
                }
        const uint32_t byte_sel = (uint32_t)t * 0x1111u + 0x4400u;   // bytes {t, t, 4+t, 4+t}
        const uint32_t meta_sel = (t & 1) ? 0x7632u : 0x5410u;
        STAMP(4);
        // Tiles go two at a time: both are multiplied, then one cross-warp sum serves both.
        const int w_end = sh.w_begin + sh.w_count;
        for (int tile = sh.w_begin; tile < w_end; tile += 2) {
            const bool two = tile + 1 < w_end;
            float acc2[2][NT][4];
#pragma unroll
            for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int h = 0; h < NT; ++h)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc2[u][h][e] = 0.f;
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                if (u == 1 && !two) break;
                float (&acc)[NT][4] = acc2[u];
                const unsigned char* base = wait_full();
                if (tile + u == sh.w_begin) STAMP(5);
                if (tile + u == sh.w_begin + 1) STAMP(6);
                if (w_active) {
                    // value bytes of block `warp`: tile warp/2, bytes 64 (warp % 2) .. +64 of the row;
                    // index bytes: tile 4 + warp/4, bytes 32 (warp % 4) .. +32
                    const unsigned char* vsub = base + (warp >> 1) * kSubTile;
                    const unsigned char* msub = base + (4 + (warp >> 2)) * kSubTile;
                    const int vo = (warp & 1) * 64, mo = (warp & 3) * 32 + 16 * (t >> 1);
                    uint4 v0[4], v1[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        v0[i] = lds128(vsub + swz(g, vo + 16 * i));
                        v1[i] = lds128(vsub + swz(g + 8, vo + 16 * i));
                    }
                    // index words of steps 0-3 come from threads 0,1 of a quad, of steps 4-7 from threads 2,3
                    const uint4 m0 = lds128(msub + swz(g, mo));
                    const uint4 m1 = lds128(msub + swz(g + 8, mo));
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        uint32_t a[4];
                        a[0] = decode_group(word_of(v0[j >> 1], (2 * j) & 3), byte_sel);
                        a[1] = decode_group(word_of(v1[j >> 1], (2 * j) & 3), byte_sel);
                        a[2] = decode_group(word_of(v0[j >> 1], (2 * j + 1) & 3), byte_sel);
                        a[3] = decode_group(word_of(v1[j >> 1], (2 * j + 1) & 3), byte_sel);
                        // metadata word: low half = row g, high half = row g+8, 16 columns each
                        uint32_t e;
                        asm("prmt.b32 %0, %1, %2, %3;" : "=r"(e)
                            : "r"(word_of(m0, j & 3)), "r"(word_of(m1, j & 3)), "r"(meta_sel));
#pragma unroll
                        for (int h = 0; h < NT; ++h) {
                            if (j < 4) mma_sp_16832<0>(acc[h], a, xf[j][h], e);
                            else       mma_sp_16832<1>(acc[h], a, xf[j][h], e);
                        }
                    }
                }
                release();
            }
            float* r0 = next_red();
            float* r1 = next_red();
            const float2 sum = block_tile_sum2<NT>(r0, r1, acc2[0], acc2[1], w_active, sh.nb);
            if (threadIdx.x < frag) {
                st_gpu(p.Ppart + ((size_t)sh.ks * tilesW + tile) * frag + threadIdx.x, slot_bits(sum.x));
                if (two) st_gpu(p.Ppart + ((size_t)sh.ks * tilesW + tile + 1) * frag + threadIdx.x, slot_bits(sum.y));
            }
        }
    }

    STAMP(7);
    // the split-K partials of an output tile are requested early: the first tile's now,
    // the others one tile ahead
    SlotBatch pb;
    const size_t p_stride = (size_t)tilesW * frag;
    if (threadIdx.x < frag && (int)blockIdx.x < tilesW)
        slots_request(pb, p.Ppart + (size_t)blockIdx.x * frag + threadIdx.x, p_stride, p.KS);

    // ------------------------------------------------ T (bf16) into shared memory
    if (p.r > 0) {
        // a thread fetches column pair jp of every token row: one batch of NT*8 entries,
        // re-requested together while some are not yet published
        const int rp = p.r_pad, pairs = rp / 2;
        for (int jp = threadIdx.x; jp < pairs; jp += kConsumerThreads) {
            uint2 e[NT * 8];
            const bool real = 2 * jp < p.r;               // padding columns are zero
#pragma unroll
            for (int m = 0; m < NT * 8; ++m) e[m] = make_uint2(0u, real ? call - 1u : call);
            for (uint32_t spins = 0;; ++spins) {
                bool all = true;
#pragma unroll
                for (int m = 0; m < NT * 8; ++m)
                    if (e[m].y != call) e[m] = ld_gpu2(p.Tfinal + (size_t)m * pairs + jp);
#pragma unroll
                for (int m = 0; m < NT * 8; ++m) all = all && e[m].y == call;
                if (all) break;
                if (spins > kPollLimit) { ok = false; break; }
            }
#pragma unroll
            for (int m = 0; m < NT * 8; ++m) *reinterpret_cast<uint32_t*>(Ts + (size_t)m * rp + 2 * jp) = e[m].x;
        }
    }
    consumer_sync();
    STAMP(8);

    // ---------------------------------------------------------------- phase Y
    for (int tile = blockIdx.x; tile < tilesW; tile += n_ctas) {
        float psum = 0.f;
        if (threadIdx.x < frag) {
            psum = slots_finish(pb, p.Ppart + (size_t)tile * frag + threadIdx.x, p_stride, p.KS, &ok);
            if (tile + n_ctas < tilesW)
                slots_request(pb, p.Ppart + (size_t)(tile + n_ctas) * frag + threadIdx.x, p_stride, p.KS);
        }
        if (tile == (int)blockIdx.x) STAMP(9);
        // every chunk of L adds into the same accumulators: one cross-warp sum per output tile
        float ytot[NT][4];
#pragma unroll
        for (int h = 0; h < NT; ++h)
#pragma unroll
            for (int e = 0; e < 4; ++e) ytot[h][e] = 0.f;
        for (int lc = 0; lc < l_chunks; ++lc) {
            const int cols = min(kLC, p.r - lc * kLC);
            const bool q_active = QA && warp * 128 < cols;
            float sc0 = 0.f, sc1 = 0.f;                   // quantized L: scales of rows g, g + 8 in the warp's group
            if (q_active) {
                const size_t grp = (size_t)((lc * kLC + warp * 128) >> 7), per_row = (size_t)((p.r + 127) >> 7);
                sc0 = __bfloat162float(p.Ls[(size_t)(tile * 16 + g) * per_row + grp]);
                sc1 = __bfloat162float(p.Ls[(size_t)(tile * 16 + g + 8) * per_row + grp]);
            }
            const bool direct = QA && p.l_direct;
            // codes of L straight from global memory (rows of r / 2 bytes, 4-byte aligned words; past r: zero)
            uint32_t dw[2][2][2] = {};
            if (direct && q_active) {
                const uint8_t* row0 = p.Lq + (size_t)(tile * 16 + g) * (size_t)(p.r / 2);
                const uint8_t* row1 = row0 + (size_t)8 * (size_t)(p.r / 2);
#pragma unroll
                for (int ss = 0; ss < 2; ++ss)
#pragma unroll
                    for (int jj = 0; jj < 2; ++jj) {
                        const int col = lc * kLC + warp * 128 + ss * 64 + jj * 32 + 8 * t;
                        if (col < p.r) {
                            dw[ss][jj][0] = __ldg(reinterpret_cast<const uint32_t*>(row0 + col / 2));
                            dw[ss][jj][1] = __ldg(reinterpret_cast<const uint32_t*>(row1 + col / 2));
                        }
                    }
            }
            const unsigned char* base = direct ? nullptr : wait_full();
            float acc[NT][4];
#pragma unroll
            for (int h = 0; h < NT; ++h)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[h][e] = 0.f;
            // warp w owns the 64-column tile w of the chunk (two 32-column blocks)
            if (q_active) {
                // quantized: the warp's group = 64 bytes of codes per row in the tile of 256 codes w / 2; codes past r read as zero
                const unsigned char* sub = base + (warp >> 1) * kSubTile;
#pragma unroll
                for (int ss = 0; ss < 2; ++ss) {
                    if (warp * 128 + ss * 64 < cols) {
#pragma unroll
                        for (int jj = 0; jj < 2; ++jj) {
                            const int kk = warp * 128 + ss * 64 + jj * 32 + 8 * t;          // column inside the chunk
                            const uint32_t wa = direct ? dw[ss][jj][0] : lds32(sub + swz(g, (warp & 1) * 64 + ss * 32 + jj * 16 + t * 4));
                            const uint32_t wb = direct ? dw[ss][jj][1] : lds32(sub + swz(g + 8, (warp & 1) * 64 + ss * 32 + jj * 16 + t * 4));
                            uint32_t a[4], c[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) { a[i] = nib_pair(wa >> (4 * i)); c[i] = nib_pair(wb >> (4 * i)); }
#pragma unroll
                            for (int h = 0; h < NT; ++h) {
                                const uint4 tb = pair_four_apart(lds128(Ts + (size_t)(g + 8 * h) * p.r_pad + lc * kLC + kk));
                                mma_16816(acc[h], a[0], c[0], a[1], c[1], tb.x, tb.y);
                                mma_16816(acc[h], a[2], c[2], a[3], c[3], tb.z, tb.w);
                            }
                        }
                    }
                }
#pragma unroll
                for (int h = 0; h < NT; ++h) {
                    ytot[h][0] = fmaf(acc[h][0], sc0, ytot[h][0]); ytot[h][1] = fmaf(acc[h][1], sc0, ytot[h][1]);
                    ytot[h][2] = fmaf(acc[h][2], sc1, ytot[h][2]); ytot[h][3] = fmaf(acc[h][3], sc1, ytot[h][3]);
                }
            } else if (!QA && warp * 64 < cols) {
                const unsigned char* sub = base + warp * kSubTile;
#pragma unroll
                for (int jj = 0; jj < 2; ++jj) {
                    const int kk = warp * 64 + jj * 32 + 8 * t;          // column inside the chunk
                    const uint4 la = lds128(sub + swz(g, jj * 64 + t * 16));   // columns past r read as zero
                    const uint4 lb = lds128(sub + swz(g + 8, jj * 64 + t * 16));
#pragma unroll
                    for (int h = 0; h < NT; ++h) {
                        const uint4 tb = lds128(Ts + (size_t)(g + 8 * h) * p.r_pad + lc * kLC + kk);
                        mma_16816(acc[h], la.x, lb.x, la.y, lb.y, tb.x, tb.y);
                        mma_16816(acc[h], la.z, lb.z, la.w, lb.w, tb.z, tb.w);
                    }
                }
            }
            if (!QA) {
#pragma unroll
                for (int h = 0; h < NT; ++h)
#pragma unroll
                    for (int e = 0; e < 4; ++e) ytot[h][e] += acc[h][e];
            }
            if (!direct) release();
        }
        const float ysum = l_chunks > 0 ? block_tile_sum<NT>(next_red(), ytot, true, kConsumerWarps) : 0.f;
        if (threadIdx.x < frag) {
            const int hq = threadIdx.x >> 5, ln = threadIdx.x & 31;
            const int h = hq >> 2, q = hq & 3;
            const int n = tile * 16 + (ln >> 2) + 8 * (q >> 1);
            const int m = 8 * h + 2 * (ln & 3) + (q & 1);
            if (m < p.b) p.Y[(size_t)m * p.d_out + n] = __float2bfloat16_rn(fmaf(psum, p.s, ysum));
        }
    }

    STAMP(10);
    if (!ok && lane == 0) flag_error(p.status, SLIM_ERR_TIMEOUT);
    consumer_sync();                                       // every poll of this CTA is over
    if (threadIdx.x == 0) atomicAdd(p.departures, 1ull);
}

// ------------------------------------------------------------------ host side
struct DecodePlan {
    int nt, KS, nblk, G, QT, r_pad, n_slots;
    size_t p_bytes, tpart_bytes, tfinal_bytes, smem;
};

static int pad_rank(int r) {
    if (r == 0) return 0;
    int rp = (r + 63) / 64 * 64;     // the last L chunk is read in whole 64-column tiles
    return rp + 32;                  // token rows 64 bytes apart modulo 128: conflict-free 16-byte reads
}

static bool shape_ok(int b, int d_out, int d_in, int r) {
    return b >= 1 && b <= 16 && d_in % 256 == 0 && d_out % 16 == 0 && r % 16 == 0 && r >= 0 && r <= kMaxDecodeRank &&
           d_in / 256 <= kMaxSlices * kConsumerWarps;
}

static bool make_plan(int b, int d_out, int d_in, int r, int ctas, DecodePlan* pl, bool qa = false) {
    if (!shape_ok(b, d_out, d_in, r)) return false;
    pl->nt = b <= 8 ? 1 : 2;
    pl->nblk = d_in / 256;
    pl->KS = ceil_div(pl->nblk, kConsumerWarps);
    pl->G = ctas / pl->KS;
    if (pl->G < 1) return false;
    int qt = 0;
    for (int k = 0; k < pl->KS; ++k) {
        const int nbk = (int)((long long)(k + 1) * pl->nblk / pl->KS) - (int)((long long)k * pl->nblk / pl->KS);
        qt += qa ? (nbk + 7) / 8 : (nbk + 1) / 2;       // R chunks of 8 blocks (quantized adapters) or 2
    }
    pl->QT = qt;
    pl->r_pad = pad_rank(r);
    const size_t frag = (size_t)pl->nt * 128 * sizeof(float);
    const size_t fixed = 1024 /* alignment slack */ + 32 * (size_t)pl->nt * 8 * 128 /* X slice */ +
                         (size_t)pl->nt * 8 * pl->r_pad * 2 + kRedBufs * kConsumerWarps * frag + (2 * kMaxSlots + 2) * 8 + 64;
    if (fixed + 3 * (size_t)kSlotBytes > kSmemBudget) return false;
    int n = (int)((kSmemBudget - fixed) / kSlotBytes);
    pl->n_slots = n > kMaxSlots ? kMaxSlots : n;
    pl->smem = (size_t)pl->n_slots * kSlotBytes + fixed;
    pl->p_bytes = (size_t)pl->KS * (d_out / 16) * frag;
    pl->tpart_bytes = (size_t)(r / 16) * pl->QT * frag;
    pl->tfinal_bytes = kTfinalBytes;
    return true;
}

int decode_query_residency(int nt) {
    int n = 0;
    cudaError_t e1, e2;
    if (nt == 1) {
        e1 = cudaFuncSetAttribute(decode_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget);
        e2 = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_kernel<1>, kDecodeThreads, kSmemBudget);
    } else {
        e1 = cudaFuncSetAttribute(decode_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget);
        e2 = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_kernel<2>, kDecodeThreads, kSmemBudget);
    }
    if (e1 != cudaSuccess || e2 != cudaSuccess) return 0;
    // the quantized-adapter instances use the same resources
    if (nt == 1) e1 = cudaFuncSetAttribute(decode_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget);
    else         e1 = cudaFuncSetAttribute(decode_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget);
    if (e1 != cudaSuccess) return 0;
    return n > 1 ? 1 : n;      // one CTA per SM: the plan sizes the grid for that
}

static int decode_ctas(int nt) {
    slim_status_t err;
    const DeviceInfo* di = device_info(&err);
    if (!di) return 148;       // sizing queries without a device assume a full B200
    return di->sm_count * (di->decode_ctas_per_sm[nt - 1] > 0 ? 1 : 0);
}

// Quantized adapters: when the rows of L's codes (r / 2 bytes) are no 16-byte multiples no tensor map can
// describe them, and the kernel reads them with plain loads.
bool decode_supports_q(int b, int d_out, int d_in, int r) {
    return r >= 16 && decode_supports(b, d_out, d_in, r);
}

bool decode_supports(int b, int d_out, int d_in, int r) {
    DecodePlan pl;
    if (b < 1 || b > 16) return false;
    return make_plan(b, d_out, d_in, r, decode_ctas(b <= 8 ? 1 : 2), &pl);
}

size_t decode_workspace_bytes(int b, int d_out, int d_in, int r) {
    // split-K partial slots and the published bf16 T; depends on the shape only, not on the device
    DecodePlan pl;
    if (!make_plan(b, d_out, d_in, r, 1 << 20, &pl)) return 0;
    return pl.p_bytes + pl.tpart_bytes + pl.tfinal_bytes;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Row-major 2-D tensor [rows][row_elems] of `esize`-byte elements, tiles of box_rows x 128 bytes.
static bool make_tile_map(CUtensorMap* map, const void* base, CUtensorMapDataType type, int esize,
                          uint64_t row_elems, uint64_t rows, int box_rows) {
    EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(tensor_map_encoder());
    if (!fn) return false;
    cuuint64_t dims[2] = {row_elems, rows};
    cuuint64_t strides[1] = {row_elems * (uint64_t)esize};
    cuuint32_t box[2] = {(cuuint32_t)(128 / esize), (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, type, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
           CUDA_SUCCESS;
}

static slim_status_t launch_decode_any(const __nv_bfloat16* X, int b, const uint8_t* vals, const uint8_t* meta,
                                       float s, const void* L, const void* R, const __nv_bfloat16* Ls, const __nv_bfloat16* Rs,
                                       int r, int d_out, int d_in, __nv_bfloat16* Y, void* ws, uint32_t* status_dev,
                                       cudaStream_t st);

slim_status_t launch_decode(const __nv_bfloat16* X, int b, const uint8_t* vals, const uint8_t* meta,
                            float s, const __nv_bfloat16* L, const __nv_bfloat16* R, int r,
                            int d_out, int d_in, __nv_bfloat16* Y, void* ws, uint32_t* status_dev,
                            cudaStream_t st)
{
    return launch_decode_any(X, b, vals, meta, s, L, R, nullptr, nullptr, r, d_out, d_in, Y, ws, status_dev, st);
}

slim_status_t launch_decode_q(const __nv_bfloat16* X, int b, const uint8_t* vals, const uint8_t* meta, float s,
                              const uint8_t* Lq, const __nv_bfloat16* Ls, const uint8_t* Rq, const __nv_bfloat16* Rs, int r,
                              int d_out, int d_in, __nv_bfloat16* Y, void* ws, uint32_t* status_dev, cudaStream_t st)
{
    if (!decode_supports_q(b, d_out, d_in, r)) return SLIM_ERR_UNSUPPORTED_SHAPE;
    return launch_decode_any(X, b, vals, meta, s, Lq, Rq, Ls, Rs, r, d_out, d_in, Y, ws, status_dev, st);
}

// Ls == nullptr: L and R are bf16 matrices; else they are the code bytes of quantized adapters.
static slim_status_t launch_decode_any(const __nv_bfloat16* X, int b, const uint8_t* vals, const uint8_t* meta,
                                       float s, const void* L, const void* R, const __nv_bfloat16* Ls, const __nv_bfloat16* Rs,
                                       int r, int d_out, int d_in, __nv_bfloat16* Y, void* ws, uint32_t* status_dev,
                                       cudaStream_t st)
{
    const bool qa = Ls != nullptr;
    slim_status_t err;
    const DeviceInfo* di = device_info(&err);
    if (!di) return err;
    DecodePlan pl;
    const int nt = b <= 8 ? 1 : 2;
    const int ctas = decode_ctas(nt);
    if (ctas < 1 || !make_plan(b, d_out, d_in, r, ctas, &pl, qa)) return SLIM_ERR_UNSUPPORTED_SHAPE;
    DecodeParams p;
    p.X = X; p.vals = vals; p.meta = meta; p.Y = Y;
    p.L = qa ? nullptr : static_cast<const __nv_bfloat16*>(L); p.R = qa ? nullptr : static_cast<const __nv_bfloat16*>(R);
    p.Ls = Ls; p.Rs = Rs;
    char* base = reinterpret_cast<char*>(ws);
    p.departures = reinterpret_cast<unsigned long long*>(base);
    p.Tfinal = reinterpret_cast<uint2*>(base + SLIM_WORKSPACE_SYNC_BYTES);
    p.Ppart = reinterpret_cast<uint32_t*>(base + SLIM_WORKSPACE_SYNC_BYTES + kTfinalBytes);
    p.Tpart = reinterpret_cast<uint32_t*>(base + SLIM_WORKSPACE_SYNC_BYTES + kTfinalBytes + pl.p_bytes);
    p.status = status_dev;
    p.s = s; p.b = b; p.r = r; p.d_out = d_out; p.d_in = d_in;
    p.KS = pl.KS; p.nblk = pl.nblk; p.G = pl.G; p.QT = pl.QT; p.r_pad = pl.r_pad;
    p.n_slots = pl.n_slots; p.chunk_blocks = qa ? 8 : 2;
    p.l_direct = qa && r % 32 != 0; p.Lq = qa ? static_cast<const uint8_t*>(L) : nullptr;
    CUtensorMap tmX, tmV, tmM, tmR, tmL;
    bool ok = make_tile_map(&tmX, X, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)d_in, (uint64_t)b, nt * 8) &&
              make_tile_map(&tmV, vals, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)d_in / 4, (uint64_t)d_out, 16) &&
              make_tile_map(&tmM, meta, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)d_in / 8, (uint64_t)d_out, 16);
    if (ok && r > 0 && qa)
        ok = make_tile_map(&tmR, R, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)d_in / 2, (uint64_t)r, 16) &&
             (r % 32 != 0 ? (tmL = tmV, true)       // not used: those codes are read with plain loads
                          : make_tile_map(&tmL, L, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)r / 2, (uint64_t)d_out, 16));
    else if (ok && r > 0)
        ok = make_tile_map(&tmR, R, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)d_in, (uint64_t)r, 16) &&
             make_tile_map(&tmL, L, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)r, (uint64_t)d_out, 16);
    else if (ok) { tmR = tmV; tmL = tmV; }       // never used when r == 0
    if (!ok) return SLIM_ERR_CUDA;
    void* args[] = {&p, &tmX, &tmV, &tmM, &tmR, &tmL};
    const dim3 grid(ctas), block(kDecodeThreads);
    const void* fn = nt == 1 ? (qa ? (const void*)decode_kernel<1, true> : (const void*)decode_kernel<1, false>)
                             : (qa ? (const void*)decode_kernel<2, true> : (const void*)decode_kernel<2, false>);
    cudaError_t e = cudaLaunchCooperativeKernel(fn, grid, block, args, pl.smem, st);
    count_launch(1);
    return e == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

}  // namespace slim

#ifdef SLIM_DECODE_TRACE
extern "C" int slim_debug_read_trace(unsigned long long* out) {
    return (int)cudaMemcpyFromSymbol(out, slim::g_trace, sizeof(slim::g_trace));
}
#endif
