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
// Data movement.  Every streamed operand travels HBM -> shared memory as TMA
// tiles (cp.async.bulk.tensor.2d, 16 rows x 128 bytes, 128-byte swizzle,
// mbarrier completion) into a ring of 16 KB slots (~190 KB in flight per SM),
// issued by one lane of a ninth, producer warp; the eight consumer warps read
// fragments from shared memory.  The producer warp also publishes the CTA's
// arrivals at the grid-wide counters (fence + atomic), so that the consumers
// never wait for a fence.  Activations live in registers as B fragments.
//
// Work split.  d_in is cut into 256-column blocks and into k-slices of <= 8
// blocks; a CTA belongs to one slice.  Each CTA first takes its share of R
// chunks (16 rows x 512 columns), then its share of 16-row weight tiles; both
// leave split-K partial tiles (fp32, MMA fragment order) in the workspace.
// Because every CTA does its R share first, T = X R^T is complete early: one
// CTA per 16 columns of T sums the partials and rounds to bf16 while the weight
// stream is still running (its ring keeps filling meanwhile).  After the weight
// phase a grid-wide counter releases the last phase, in which every CTA
// finishes 16-row output tiles:  Y = s * sum(partials) + T L^T, with the L
// rows already prefetched into the ring.  All waits on other CTAs are bounded
// spins (the launch is cooperative, so all CTAs are resident); an expired wait
// sets SLIM_ERR_TIMEOUT and the kernel runs on to its end.  Reductions have a
// fixed order: results are bit-identical from run to run.
#include <cuda.h>
#include "common.cuh"

namespace slim {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kDecodeThreads = kConsumerThreads + 32;     // + producer warp
constexpr int kMaxDecodeRank = 3072;
constexpr int kMaxSlots = 16;
constexpr uint32_t kSpinLimit = 1u << 22;                  // global counters (each poll sleeps >= 20 ns)
constexpr uint32_t kMbarSpinLimit = 1u << 26;              // shared-memory barriers
constexpr int kRChunkCols = 512;                           // columns of one R chunk
constexpr int kLChunkCols = 512;                           // columns (of r) of one L chunk
constexpr size_t kSmemBudget = 227 * 1024;
enum { EV_R = 0, EV_T = 1, EV_W = 2 };                   // consumer -> producer events

// Synchronisation words in the first bytes of the workspace.
enum { SYNC_R = 0, SYNC_T = 1, SYNC_W = 2, SYNC_DEPART = 3 };

struct DecodeParams {
    const __nv_bfloat16* X; const uint8_t* vals; const uint8_t* meta;
    const __nv_bfloat16* L; const __nv_bfloat16* R; __nv_bfloat16* Y;
    float* Ppart;              // [KS][tilesW][frag]
    float* Tpart;              // [tilesR][QT][frag]
    __nv_bfloat16* Tfinal;     // [NT*8][r_pad]
    uint32_t* sync; uint32_t* status;
    float s;
    int b, r, d_out, d_in;
    int KS, nblk, G, QT, r_pad;
    int n_slots;
};
constexpr int kSubTile = 2048;                             // one TMA box: 16 rows x 128 bytes
constexpr int kSlotBytes = 8 * kSubTile;

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
// One TMA tile (16 rows x 128 bytes of the tensor behind `tmap`, starting at
// element column x, row y) into shared memory; completion in bytes on `bar`.
__device__ __forceinline__ void tma_tile(void* dst, const CUtensorMap* tmap, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 :: "r"(smem_u32(dst)), "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return done != 0;
}
// Byte address inside a 128-byte-swizzled tile of 16 rows: the 16-byte chunk
// index is XOR-ed with the row number modulo 8.
__device__ __forceinline__ uint32_t swz(int row, int byte_off) {
    return (uint32_t)(row * 128 + ((((byte_off >> 4) ^ row) & 7) << 4) + (byte_off & 15));
}
__device__ __forceinline__ void consumer_sync() {          // the eight consumer warps only
    asm volatile("bar.sync 1, %0;" :: "n"(kConsumerThreads) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint4 lds128(const void* p) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(smem_u32(p)));
    return v;
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

// ------------------------------------------------------------ work split
// Everything below is computed identically by the producer and the consumers.
struct Share {
    int ks, grp;             // k-slice and position inside the slice's CTA group (-1: no phase-1 work)
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
    sh.Qk = (sh.nb + 1) / 2;
    int qoff = 0;
    for (int k = 0; k < sh.ks; ++k) {
        const int nbk = (int)((long long)(k + 1) * p.nblk / p.KS) - (int)((long long)k * p.nblk / p.KS);
        qoff += (nbk + 1) / 2;
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

template <int NT>
__global__ void __launch_bounds__(kDecodeThreads, 1)
decode_kernel(const DecodeParams p, const __grid_constant__ CUtensorMap tmV,
              const __grid_constant__ CUtensorMap tmM, const __grid_constant__ CUtensorMap tmR,
              const __grid_constant__ CUtensorMap tmL)
{
    constexpr int frag = NT * 128;
    extern __shared__ unsigned char smem_raw[];
    // layout (ring first, 1024-byte aligned for the swizzle): ring slots | Ts | red x2 | barriers | flags
    unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __nv_bfloat16* Ts = reinterpret_cast<__nv_bfloat16*>(ring + (size_t)p.n_slots * kSlotBytes);
    float* red_base = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(Ts) + (size_t)NT * 8 * p.r_pad * 2);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(red_base + 2 * kConsumerWarps * frag);
    uint64_t* empty_bar = full_bar + kMaxSlots;
    uint64_t* event_bar = empty_bar + kMaxSlots;            // EV_R, EV_T, EV_W
    volatile uint32_t* flags = reinterpret_cast<volatile uint32_t*>(event_bar + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int tilesW = p.d_out / 16, tilesR = p.r / 16;
    const int n_ctas = gridDim.x;
    const Share sh = make_share(p, blockIdx.x);
    const int n_slots = p.n_slots;
    const int l_chunks = p.r > 0 ? ceil_div(p.r, kLChunkCols) : 0;
    int t_mine = 0;                                          // 16-column pieces of T this CTA sums
    if (p.r > 0) for (int jt = blockIdx.x; jt < tilesR; jt += n_ctas) ++t_mine;

    if (threadIdx.x == 0) {
        for (int i = 0; i < n_slots; ++i) { mbar_init(&full_bar[i], 1); mbar_init(&empty_bar[i], kConsumerWarps); }
        for (int i = 0; i < 3; ++i) mbar_init(&event_bar[i], kConsumerWarps);
        flags[0] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == kConsumerWarps) {
        // ============================ producer warp ============================
        // Lane 0 runs the ring protocol and publishes arrivals; lanes 0-7 each issue
        // one 2 KB tile of a chunk (a single thread can start only ~6 TMA loads per
        // microsecond, eight threads in parallel about 20).
        uint32_t it = 0;
        bool ok = true;
        bool pend_r = p.r > 0, pend_t = t_mine > 0, pend_w = true;
        // Publish the CTA's arrivals: the consumers signal an event after their
        // stores; lane 0 makes them visible device-wide and bumps the counter.
        auto service = [&]() {
            if (pend_r && mbar_test(&event_bar[EV_R], 0)) { __threadfence(); atomicAdd(&p.sync[SYNC_R], 1u); pend_r = false; }
            if (pend_t && mbar_test(&event_bar[EV_T], 0)) { __threadfence(); atomicAdd(&p.sync[SYNC_T], (uint32_t)t_mine); pend_t = false; }
            if (pend_w && mbar_test(&event_bar[EV_W], 0)) { __threadfence(); atomicAdd(&p.sync[SYNC_W], 1u); pend_w = false; }
        };
        // Returns the slot (all lanes) once it is free and its full barrier is armed.
        auto acquire = [&](uint32_t bytes) -> int {
            const int slot = it % n_slots;
            if (lane == 0) {
                service();
                if (it >= (uint32_t)n_slots) {
                    const uint32_t parity = ((it / n_slots) & 1) ^ 1;
                    uint32_t spins = 0;
                    while (!mbar_test(&empty_bar[slot], parity)) {
                        service();
                        if (++spins > kMbarSpinLimit) { ok = false; break; }
                    }
                }
                mbar_arrive_expect_tx(&full_bar[slot], bytes);
            }
            __syncwarp();
            ++it;
            return slot;
        };
        // ---- R chunks: 16 rows x (256 or 512) columns of bf16 = 4 or 8 tiles of 64 columns
        for (int u = sh.r_begin; u < sh.r_begin + sh.r_count; ++u) {
            const int tile = u / sh.Qk, q = u % sh.Qk;
            const int cols = min(kRChunkCols, sh.nb * 256 - q * kRChunkCols);
            const int n_sub = cols / 64;
            const int slot = acquire((uint32_t)n_sub * kSubTile);
            if (lane < n_sub)
                tma_tile(ring + (size_t)slot * kSlotBytes + lane * kSubTile, &tmR,
                         sh.blk_begin * 256 + q * kRChunkCols + 64 * lane, tile * 16, &full_bar[slot]);
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
        for (int tile = blockIdx.x; tile < tilesW && p.r > 0; tile += n_ctas) {
            for (int lc = 0; lc < l_chunks; ++lc) {
                const int cols = min(kLChunkCols, p.r - lc * kLChunkCols);
                const int n_sub = ceil_div(cols, 64);
                const int slot = acquire((uint32_t)n_sub * kSubTile);
                if (lane < n_sub)
                    tma_tile(ring + (size_t)slot * kSlotBytes + lane * kSubTile, &tmL,
                             lc * kLChunkCols + 64 * lane, tile * 16, &full_bar[slot]);
            }
        }
        // ---- remaining arrivals
        if (lane == 0) {
            for (uint32_t spins = 0; (pend_r || pend_t || pend_w); ++spins) {
                service();
                if (spins > kMbarSpinLimit) { ok = false; break; }
            }
            if (!ok) flag_error(p.status, SLIM_ERR_TIMEOUT);
        }
        return;      // the consumers wait for every tile this warp requested before they leave
    }

    // ================================ consumer warps ================================
    uint32_t it = 0;
    int red_buf = 0;
    bool ok = true;
    auto wait_full = [&]() -> unsigned char* {
        const int slot = it % n_slots;
        ok = mbar_wait(&full_bar[slot], (it / n_slots) & 1) && ok;
        return ring + (size_t)slot * kSlotBytes;
    };
    auto release = [&]() {
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[it % n_slots]);
        ++it;
    };
    auto next_red = [&]() -> float* {
        float* r = red_base + red_buf * kConsumerWarps * frag;
        red_buf ^= 1;
        return r;
    };
    // Every warp's global stores are done: tell the producer warp to publish them.
    auto signal = [&](int ev) {
        __syncwarp();
        if (lane == 0) mbar_arrive(&event_bar[ev]);
    };
    // Thread 0 waits (bounded) for a grid-wide counter; all consumer warps leave together.
    auto wait_counter = [&](int which, uint32_t target) {
        if (threadIdx.x == 0) {
            bool reached = false;
            for (uint32_t i = 0; i < kSpinLimit; ++i) {
                if (ld_acquire(&p.sync[which]) >= target) { reached = true; break; }
                __nanosleep(20);
            }
            if (!reached) flag_error(p.status, SLIM_ERR_TIMEOUT);
        }
        consumer_sync();
    };

    // activations as sparse B fragments for the weight phase: step j, n-tile h, register i
    // holds X[g + 8h][slice + 256 warp + 32 j + 2 t + 8 i .. +1].  Requested first: they
    // are needed last, after the R chunks.
    const bool w_active = warp < sh.nb && sh.w_count > 0;
    uint32_t xf[8][NT][4];
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int h = 0; h < NT; ++h)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = g + 8 * h;
                xf[j][h][i] = (w_active && row < p.b)
                    ? __ldg(reinterpret_cast<const uint32_t*>(p.X + (size_t)row * p.d_in + (size_t)(sh.blk_begin + warp) * 256 + 32 * j + 2 * t + 8 * i))
                    : 0u;
            }

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
                    const int row = g + 8 * h;
                    const int col = q * kRChunkCols + warp * 64 + jj * 32;
                    xd[q][jj][h] = (col < sh.nb * 256 && row < p.b)
                        ? __ldg(reinterpret_cast<const uint4*>(p.X + (size_t)row * p.d_in + (size_t)sh.blk_begin * 256 + col + 8 * t))
                        : make_uint4(0, 0, 0, 0);
                }
        for (int u = sh.r_begin; u < sh.r_begin + sh.r_count; ++u) {
            const int tile = u / sh.Qk, q = u % sh.Qk;
            const int cols = min(kRChunkCols, sh.nb * 256 - q * kRChunkCols);
            const bool active = warp * 64 < cols;
            const unsigned char* base = wait_full();
            float acc[NT][4];
#pragma unroll
            for (int h = 0; h < NT; ++h)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[h][e] = 0.f;
            if (active) {
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
            const float sum = block_tile_sum<NT>(next_red(), acc, active, min(kConsumerWarps, cols / 64));
            if (threadIdx.x < frag)
                p.Tpart[((size_t)tile * p.QT + sh.qoff + q) * frag + threadIdx.x] = sum;
        }
    }
    if (p.r > 0) signal(EV_R);

    // T reduction duty: CTA c owns the 16-column pieces jt = c, c + n_ctas, ...
    bool t_pending = t_mine > 0;
    auto reduce_t = [&]() {
        for (int jt = blockIdx.x; jt < tilesR; jt += n_ctas) {
            if (threadIdx.x < frag) {
                const float* src = p.Tpart + (size_t)jt * p.QT * frag + threadIdx.x;
                float sum = 0.f;
#pragma unroll 8
                for (int sl = 0; sl < p.QT; ++sl) sum += __ldcg(src + (size_t)sl * frag);
                const int hq = threadIdx.x >> 5, ln = threadIdx.x & 31;
                const int h = hq >> 2, q = hq & 3;
                const int j = jt * 16 + (ln >> 2) + 8 * (q >> 1);
                const int m = 8 * h + 2 * (ln & 3) + (q & 1);
                p.Tfinal[(size_t)m * p.r_pad + j] = __float2bfloat16_rn(sum);
            }
        }
        signal(EV_T);
        t_pending = false;
    };

    // ---------------------------------------------------------------- phase W
    if (sh.w_count > 0) {
        const uint32_t byte_sel = (uint32_t)t * 0x1111u + 0x4400u;   // bytes {t, t, 4+t, 4+t}
        const uint32_t meta_sel = (t & 1) ? 0x7632u : 0x5410u;
        // the CTAs with reduction duty look at the R counter once per tile; the load is
        // issued one tile ahead so that its latency is never waited for
        uint32_t polled = 0;
        if (t_pending && threadIdx.x == 0) polled = ld_acquire(&p.sync[SYNC_R]);
        for (int tile = sh.w_begin; tile < sh.w_begin + sh.w_count; ++tile) {
            if (t_pending) {
                if (threadIdx.x == 0) flags[0] = polled >= (uint32_t)n_ctas ? 1u : 0u;
                consumer_sync();
                const bool ready = flags[0] != 0;
                consumer_sync();
                if (ready) reduce_t();
                else if (threadIdx.x == 0) polled = ld_acquire(&p.sync[SYNC_R]);
            }
            const unsigned char* base = wait_full();
            float acc[NT][4];
#pragma unroll
            for (int h = 0; h < NT; ++h)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[h][e] = 0.f;
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
            const float sum = block_tile_sum<NT>(next_red(), acc, w_active, sh.nb);
            if (threadIdx.x < frag)
                p.Ppart[((size_t)sh.ks * tilesW + tile) * frag + threadIdx.x] = sum;
        }
    }
    signal(EV_W);

    // ------------------------------------------------ T: finish, then fetch
    if (p.r > 0) {
        if (t_pending) { wait_counter(SYNC_R, (uint32_t)n_ctas); reduce_t(); }
        wait_counter(SYNC_T, (uint32_t)tilesR);
        const int rp = p.r_pad;
        for (int idx = threadIdx.x; idx < NT * 8 * (rp / 8); idx += kConsumerThreads) {
            const int m = idx / (rp / 8), c8 = (idx % (rp / 8)) * 8;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (c8 < p.r) v = __ldcg(reinterpret_cast<const uint4*>(p.Tfinal + (size_t)m * rp + c8));
            *reinterpret_cast<uint4*>(Ts + (size_t)m * rp + c8) = v;
        }
    }
    wait_counter(SYNC_W, (uint32_t)n_ctas);              // ends with a consumer_sync: Ts is visible

    // ---------------------------------------------------------------- phase Y
    auto load_psum = [&](int tile) -> float {
        float v = 0.f;
        if (threadIdx.x < frag && tile < tilesW) {
            const float* src = p.Ppart + (size_t)tile * frag + threadIdx.x;
#pragma unroll 4
            for (int ks = 0; ks < p.KS; ++ks) v += __ldcg(src + (size_t)ks * tilesW * frag);
        }
        return v;
    };
    float psum_next = load_psum(blockIdx.x);
    for (int tile = blockIdx.x; tile < tilesW; tile += n_ctas) {
        const float psum = psum_next;
        psum_next = load_psum(tile + n_ctas);             // one tile ahead
        float ysum = 0.f;
        for (int lc = 0; lc < l_chunks; ++lc) {
            const int cols = min(kLChunkCols, p.r - lc * kLChunkCols);
            const unsigned char* base = wait_full();
            float acc[NT][4];
#pragma unroll
            for (int h = 0; h < NT; ++h)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[h][e] = 0.f;
            // warp w owns the 64-column tile w of the chunk (two 32-column blocks)
            if (warp * 64 < cols) {
                const unsigned char* sub = base + warp * kSubTile;
#pragma unroll
                for (int jj = 0; jj < 2; ++jj) {
                    const int kk = warp * 64 + jj * 32 + 8 * t;          // column inside the chunk
                    const uint4 la = lds128(sub + swz(g, jj * 64 + t * 16));   // columns past r read as zero
                    const uint4 lb = lds128(sub + swz(g + 8, jj * 64 + t * 16));
#pragma unroll
                    for (int h = 0; h < NT; ++h) {
                        const uint4 tb = lds128(Ts + (size_t)(g + 8 * h) * p.r_pad + lc * kLChunkCols + kk);
                        mma_16816(acc[h], la.x, lb.x, la.y, lb.y, tb.x, tb.y);
                        mma_16816(acc[h], la.z, lb.z, la.w, lb.w, tb.z, tb.w);
                    }
                }
            }
            release();
            ysum += block_tile_sum<NT>(next_red(), acc, true, kConsumerWarps);
        }
        if (threadIdx.x < frag) {
            const int hq = threadIdx.x >> 5, ln = threadIdx.x & 31;
            const int h = hq >> 2, q = hq & 3;
            const int n = tile * 16 + (ln >> 2) + 8 * (q >> 1);
            const int m = 8 * h + 2 * (ln & 3) + (q & 1);
            if (m < p.b) p.Y[(size_t)m * p.d_out + n] = __float2bfloat16_rn(fmaf(psum, p.s, ysum));
        }
    }

    // the last CTA to leave puts the counters back to zero for the next call
    if (!ok && lane == 0) flag_error(p.status, SLIM_ERR_TIMEOUT);
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(&p.sync[SYNC_DEPART], 1u) == (uint32_t)n_ctas - 1) {
            p.sync[SYNC_R] = 0u; p.sync[SYNC_T] = 0u; p.sync[SYNC_W] = 0u; p.sync[SYNC_DEPART] = 0u;
            __threadfence();
        }
    }
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
    return b >= 1 && b <= 16 && d_in % 256 == 0 && d_out % 16 == 0 && r % 16 == 0 && r >= 0 && r <= kMaxDecodeRank;
}

static bool make_plan(int b, int d_out, int d_in, int r, int ctas, DecodePlan* pl) {
    if (!shape_ok(b, d_out, d_in, r)) return false;
    pl->nt = b <= 8 ? 1 : 2;
    pl->nblk = d_in / 256;
    pl->KS = ceil_div(pl->nblk, kConsumerWarps);
    pl->G = ctas / pl->KS;
    if (pl->G < 1) return false;
    int qt = 0;
    for (int k = 0; k < pl->KS; ++k) {
        const int nbk = (int)((long long)(k + 1) * pl->nblk / pl->KS) - (int)((long long)k * pl->nblk / pl->KS);
        qt += (nbk + 1) / 2;
    }
    pl->QT = qt;
    pl->r_pad = pad_rank(r);
    const size_t frag = (size_t)pl->nt * 128 * sizeof(float);
    const size_t fixed = 1024 /* alignment slack */ + (size_t)pl->nt * 8 * pl->r_pad * 2 + 2 * kConsumerWarps * frag +
                         (2 * kMaxSlots + 4) * 8 + 64;
    if (fixed + 2 * (size_t)kSlotBytes > kSmemBudget) return false;
    int n = (int)((kSmemBudget - fixed) / kSlotBytes);
    pl->n_slots = n > kMaxSlots ? kMaxSlots : n;
    pl->smem = (size_t)pl->n_slots * kSlotBytes + fixed;
    pl->p_bytes = (size_t)pl->KS * (d_out / 16) * frag;
    pl->tpart_bytes = (size_t)(r / 16) * pl->QT * frag;
    pl->tfinal_bytes = ((size_t)pl->nt * 8 * pl->r_pad * 2 + 255) / 256 * 256;
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
    return n > 1 ? 1 : n;      // one CTA per SM: the plan sizes the grid for that
}

static int decode_ctas(int nt) {
    slim_status_t err;
    const DeviceInfo* di = device_info(&err);
    if (!di) return 148;       // sizing queries without a device assume a full B200
    return di->sm_count * (di->decode_ctas_per_sm[nt - 1] > 0 ? 1 : 0);
}

bool decode_supports(int b, int d_out, int d_in, int r) {
    DecodePlan pl;
    if (b < 1 || b > 16) return false;
    return make_plan(b, d_out, d_in, r, decode_ctas(b <= 8 ? 1 : 2), &pl);
}

size_t decode_workspace_bytes(int b, int d_out, int d_in, int r) {
    // split-K partial tiles and the bf16 T; depends on the shape only, not on the device
    DecodePlan pl;
    if (!make_plan(b, d_out, d_in, r, 1 << 20, &pl)) return 0;
    return pl.p_bytes + pl.tpart_bytes + pl.tfinal_bytes;
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// Row-major 2-D tensor [rows][row_elems] of `esize`-byte elements, tiles of 16 rows x 128 bytes.
static bool make_tile_map(CUtensorMap* map, const void* base, CUtensorMapDataType type, int esize,
                          uint64_t row_elems, uint64_t rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {row_elems, rows};
    cuuint64_t strides[1] = {row_elems * (uint64_t)esize};
    cuuint32_t box[2] = {(cuuint32_t)(128 / esize), 16};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, type, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
           CUDA_SUCCESS;
}

slim_status_t launch_decode(const __nv_bfloat16* X, int b, const uint8_t* vals, const uint8_t* meta,
                            float s, const __nv_bfloat16* L, const __nv_bfloat16* R, int r,
                            int d_out, int d_in, __nv_bfloat16* Y, void* ws, uint32_t* status_dev,
                            cudaStream_t st)
{
    slim_status_t err;
    const DeviceInfo* di = device_info(&err);
    if (!di) return err;
    DecodePlan pl;
    const int nt = b <= 8 ? 1 : 2;
    const int ctas = decode_ctas(nt);
    if (ctas < 1 || !make_plan(b, d_out, d_in, r, ctas, &pl)) return SLIM_ERR_UNSUPPORTED_SHAPE;
    DecodeParams p;
    p.X = X; p.vals = vals; p.meta = meta; p.L = L; p.R = R; p.Y = Y;
    char* base = reinterpret_cast<char*>(ws);
    p.sync = reinterpret_cast<uint32_t*>(base);
    p.Ppart = reinterpret_cast<float*>(base + SLIM_WORKSPACE_SYNC_BYTES);
    p.Tpart = reinterpret_cast<float*>(base + SLIM_WORKSPACE_SYNC_BYTES + pl.p_bytes);
    p.Tfinal = reinterpret_cast<__nv_bfloat16*>(base + SLIM_WORKSPACE_SYNC_BYTES + pl.p_bytes + pl.tpart_bytes);
    p.status = status_dev;
    p.s = s; p.b = b; p.r = r; p.d_out = d_out; p.d_in = d_in;
    p.KS = pl.KS; p.nblk = pl.nblk; p.G = pl.G; p.QT = pl.QT; p.r_pad = pl.r_pad;
    p.n_slots = pl.n_slots;
    CUtensorMap tmV, tmM, tmR, tmL;
    bool ok = make_tile_map(&tmV, vals, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)d_in / 4, (uint64_t)d_out) &&
              make_tile_map(&tmM, meta, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)d_in / 8, (uint64_t)d_out);
    if (ok && r > 0)
        ok = make_tile_map(&tmR, R, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)d_in, (uint64_t)r) &&
             make_tile_map(&tmL, L, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)r, (uint64_t)d_out);
    else if (ok) { tmR = tmV; tmL = tmV; }       // never used when r == 0
    if (!ok) return SLIM_ERR_CUDA;
    void* args[] = {&p, &tmV, &tmM, &tmR, &tmL};
    const dim3 grid(ctas), block(kDecodeThreads);
    cudaError_t e = nt == 1
        ? cudaLaunchCooperativeKernel((const void*)decode_kernel<1>, grid, block, args, pl.smem, st)
        : cudaLaunchCooperativeKernel((const void*)decode_kernel<2>, grid, block, args, pl.smem, st);
    count_launch(1);
    return e == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

}  // namespace slim
