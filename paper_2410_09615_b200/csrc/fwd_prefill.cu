// Prefill-phase forward (many tokens): tcgen05 tensor cores with the accumulator
// in tensor memory.
//
// One CTA computes a 128 (output rows) x N (tokens; N = 256, or 64 for small problems) tile of
//     out[token][row] = scale * ( sum_k W[row][k] X[token][k]  +  sum_j A2[row][j] B2[token][j] )
// in two chained phases that accumulate into the same TMEM tile:
//   phase 1 (sparse): W is the packed int4 2:4 weight.  TMA brings 128 rows of value
//       bytes and index bytes plus the X tile; eight converter warps (two groups on
//       alternate stages, one thread per weight row) expand nibbles to exact bf16 into the
//       64-byte-swizzled K-major layout the MMA reads, and write the 2:4 index words into
//       tensor memory; one thread issues tcgen05.mma.sp (kind::f16, bf16 x bf16 -> fp32).
//   phase 2 (dense): A2 and B2 are bf16 matrices brought by TMA as they are; the same
//       thread issues tcgen05.mma into the same accumulator.
// The layer forward is two or three launches:
//   T' = (X R^T) / s          phase 2 only (A2 = R, B2 = X, scale 1/s), bf16 into the workspace.
//                             The product has few tiles, so K is split over blockIdx.z; the
//                             slices write fp32 partial tiles and a small kernel adds them in a
//                             fixed order (one slice: bf16 directly, no second launch).
//   Y  = s * (X Q^T + T' L^T) phase 1 then phase 2 (A2 = L, B2 = T', scale s)
// so the adapter product and the scale are fused into the tile loop and the epilogue.
//
// Index words in tensor memory (one 32-bit column per MMA of 32 weight columns): lane
// l holds 16 of the 32 columns (half (l / 8) % 2) of two rows, row l & ~8 in bits
// 0-15 and row l | 8 in bits 16-31; the MMA addresses an even column pair and a
// selector bit of the instruction descriptor picks the column.  A 32-bit word of the
// packed index array is one row's 32 columns, so a converter thread swaps one
// half-word with the thread eight rows away and stores the result.
// Source of the layout: PTX ISA, "tcgen05.mma.sp" -- "Sparse matrices" / "Sparsity selector" for
// kind::f16 (which bits of the metadata columns in tensor memory describe which chunk of A, and
// how the selector picks a column of a pair); the one-hot and exact-integer tests check it.
//
// Pipeline.  A ring of stages {B: token rows x 128 bytes, A: 8 KB (16 KB in the dense-only
// launch)}; a sparse stage is 64 weight columns (two MMAs of K = 32), a dense stage 32 columns
// (two MMAs of K = 16; 64 columns in the dense-only launch).  The packed value and index bytes
// travel separately, 256 columns (4 stages) per TMA tile, through a ring of their own.
// Warps: 0-7 converters, then epilogue; 8 and 10 token tiles of even / odd stages (with the A2
// tile in phase 2); 9 MMA issue; 11 packed tiles.
// mbarriers: b_full / pk_full (TMA bytes landed), conv_done (converters finished a stage),
// empty / pk_empty (tcgen05.commit: the MMAs that read the stage are complete; converters
// done with a packed slot), acc_full.
// Measured on B200 and built into the loops below: a barrier operation is served per thread
// (a warp-wide try_wait or 32 arrivals cost 32 times one); the answer of a try_wait takes about
// 200 cycles even when the phase is long complete, so waits that follow each other are asked
// together; a lane left at a warp barrier while another lane of its warp spins costs some hundred
// nanoseconds per iteration; one MMA costs at least the 128 cycles its 128-row A operand takes to
// load, whatever N.  With one CTA per tile a stage takes about 320 ns: its slot's next token tile
// is requested ~600 ns after the MMAs that free the slot were issued and lands ~900 ns later, over
// the 5 stages that fit in shared memory.
// Every wait is bounded; an expired one sets SLIM_ERR_TIMEOUT and the kernel runs on.
#include <atomic>
#include <cuda.h>
#include "common.cuh"

namespace slim {

constexpr int kPM = 128;            // output rows per CTA (MMA M)
constexpr int kPBK = 64;            // columns per stage, both phases
constexpr int kPkStages = 4;        // stages covered by one packed tile (256 weight columns)
constexpr int kConvWarps = 8;       // warps 0-7 converters / epilogue
constexpr int kWarpXEven = 8, kWarpMma = 9, kWarpXOdd = 10, kWarpPk = 11;
constexpr int kPThreads = 32 * 12;
constexpr int kATile = kPM * 128;               // 16 KB: 128 rows x 128 bytes (dense phase)
constexpr int kValsTile = kPM * (kPkStages * kPBK / 4);     // 8 KB: 64 value bytes per row
constexpr int kMetaTile = kPM * (kPkStages * kPBK / 8);     // 4 KB: 32 index bytes per row
constexpr int kPkSlotBytes = kValsTile + kMetaTile;
constexpr uint32_t kPSpinLimit = 1u << 21;

// TWO = a pair of CTAs (cluster of 2 along the row tiles) shares one token tile: each CTA
// loads half of it and one cta_group::2 MMA of shape 256 x N, issued by the even CTA,
// drives both tensor cores.  Halves the token-tile traffic per CTA and leaves room for
// more stages.
// PRE = the dense-only launch (T' product): no packed tiles, so the room goes to more stages.
template <int N, bool TWO, bool PRE = false> struct PfCfg {
    static constexpr int kBRows = TWO ? N / 2 : N;                          // token rows this CTA loads
    static constexpr int kBTile = kBRows * 128;
    // A region of a stage: the expanded weight tile needs 8 KB.  The main kernels' dense stages are
    // 32 columns wide so that their A2 tile fits there too: a smaller stage means more stages in
    // flight, and the loop is bound by the latency of the token tile.  The dense-only launch
    // has no expanded tiles and keeps 64-column stages.
    static constexpr int kARegion = PRE ? kATile : kATile / 2;
    static constexpr int kDK = PRE ? 64 : 32;                               // columns of a dense stage
    static constexpr int kStages = PRE ? (N >= 256 ? 4 : 8) : (TWO ? 7 : (N >= 256 ? 5 : 8));
    // Packed tiles come from HBM (latency of a microsecond or two): the ring holds what fits.
    static constexpr int kPkSlots = PRE ? 1 : (TWO ? 4 : (N >= 256 ? 2 : 7));
    static constexpr int kStageBytes = kBTile + kARegion;
    static constexpr int kECol = N;                                         // index words: N + 4 * stage + mma
    static constexpr int kTmemCols = N >= 256 ? 512 : (N >= 128 ? 256 : 128);
    static constexpr size_t kSmem = 1024 + (size_t)kStages * kStageBytes + kPkSlots * kPkSlotBytes + 1024;
};

struct PrefillParams {
    __nv_bfloat16* out;     // [tokens][ldo]
    int ldo;
    int m_total;            // valid output rows
    int b;                  // valid tokens
    int n1, n2;             // stages of the sparse and of the dense phase
    float scale;
    uint32_t* status;
    // dense-only launch split along K over blockIdx.z: slice z covers `k_per` stages from z * k_per and
    // writes its fp32 partial tile to part[z][token][ldo] (part == nullptr: one slice, bf16 to out)
    float* part;
    int k_per;
};

// Optional timeline: built with -DSLIM_PREFILL_TRACE, one thread per warp role of the first
// CTAs records the global timer around its waits for the first 48 stages.
#ifdef SLIM_PREFILL_TRACE
#ifndef SLIM_PTRACE_PRE
#define SLIM_PTRACE_PRE 0          // 1: stamp the dense-only launch instead of the main one
#endif
__device__ unsigned long long g_ptrace[8][6][48];
#define PSTAMP(role, it) do { if (PRE == (SLIM_PTRACE_PRE != 0) && blockIdx.z == 0 && blockIdx.x + gridDim.x * blockIdx.y < 8 && (it) < 48) { unsigned long long t_; \
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); g_ptrace[blockIdx.x + gridDim.x * blockIdx.y][role][it] = t_; } } while (0)
#else
#define PSTAMP(role, it) do { } while (0)
#endif

namespace pf {

__device__ __forceinline__ uint32_t s32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(s32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(s32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(s32(bar)), "r"(bytes) : "memory");
}
// Bounded wait.  The first wait of a CTA that expires raises `*abort_flag`; every later
// wait of the CTA then gives up at once, so a broken pipeline costs one time-out, not many.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag) {
    const uint32_t addr = s32(bar);
    for (uint32_t it = 0; it < kPSpinLimit; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1u;
    return false;
}
__device__ __forceinline__ void tma_tile(void* dst, const CUtensorMap* tmap, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 :: "r"(s32(dst)), "l"(tmap), "r"(x), "r"(y), "r"(s32(bar)) : "memory");
}

// Shared-memory matrix descriptor: K-major tile of 128-byte rows, 128-byte swizzle,
// 8-row groups 1024 bytes apart (descriptor version 1).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Same with 64-byte rows and 64-byte swizzle (8-row groups 512 bytes apart).
__device__ __forceinline__ uint64_t smem_desc64(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(512 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)4 << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, both K-major.
__host__ __device__ constexpr uint32_t idesc_bf16(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ void mma_dense(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// A holds the two kept values of every group of four; e_tmem addresses the index words.
__device__ __forceinline__ void mma_sparse(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t e_tmem,
                                           uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::1.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}"
        :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(e_tmem), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(s32(bar)) : "memory");
}
// ---- CTA-pair variants
__device__ __forceinline__ void mma_dense2(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_sparse2(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t e_tmem,
                                            uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}"
        :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(e_tmem), "r"(idesc), "r"(accumulate) : "memory");
}
// Address of the same shared-memory object in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t peer_addr(const void* p, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(s32(p)), "r"(rank));
    return r;
}
// Completion of this thread's earlier MMAs arrives on a barrier given by cluster address.
__device__ __forceinline__ void mma_commit2(uint32_t cluster_bar_addr) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(cluster_bar_addr) : "memory");
}
// Arrival on a barrier of another CTA of the cluster, ordered like a CTA-local arrival.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_bar_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" :: "r"(cluster_bar_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" :: "r"(cluster_bar_addr) : "memory");
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag) {
    const uint32_t addr = s32(bar);
    for (uint32_t it = 0; it < kPSpinLimit; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1u;
    return false;
}
// One try_wait, no loop.  `cluster`: acquire at cluster scope (arrivals came from the other CTA).
__device__ __forceinline__ uint32_t mbar_try(uint64_t* bar, uint32_t parity, bool cluster) {
    uint32_t done;
    if (cluster)
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(s32(bar)), "r"(parity) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(s32(bar)), "r"(parity) : "memory");
    return done;
}
// The same question without waiting (try_wait holds the thread for a while when the answer is no).
__device__ __forceinline__ uint32_t mbar_test(uint64_t* bar, uint32_t parity, bool cluster) {
    uint32_t done;
    if (cluster)
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(s32(bar)), "r"(parity) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(s32(bar)), "r"(parity) : "memory");
    return done;
}
// Bounded wait for several barriers at once.  A try_wait takes about 200 cycles to answer even when
// the phase is long complete, so waits that follow each other are asked together, not in turn.
__device__ __forceinline__ bool mbar_wait_all(uint64_t* b0, uint32_t p0, bool c0, uint64_t* b1, uint32_t p1, bool c1,
                                              uint64_t* b2, uint32_t p2, bool c2, volatile uint32_t* abort_flag) {
    for (uint32_t it = 0; it < kPSpinLimit; ++it) {
        const uint32_t d0 = b0 ? mbar_try(b0, p0, c0) : 1u;
        const uint32_t d1 = b1 ? mbar_try(b1, p1, c1) : 1u;
        const uint32_t d2 = b2 ? mbar_try(b2, p2, c2) : 1u;
        if (d0 & d1 & d2) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1u;
    return false;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Two int4 codes of byte `T` of w -> exact bf16x2: nibble ^ 8 in the mantissa of 128.0
// is 128 + (v + 8); subtracting 136 leaves v in [-8, 7].
template <int T>
__device__ __forceinline__ uint32_t nib2bf16(uint32_t w, uint32_t w_shr4) {
    uint32_t x, y;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(x) : "r"(w), "r"(w_shr4), "n"(T * 0x1111 + 0x4400));
    asm("lop3.b32 %0, %1, %2, %3, 0x6a;" : "=r"(y) : "r"(x), "r"(0x000F000Fu), "r"(0x43084308u));
    __nv_bfloat162 v = *reinterpret_cast<__nv_bfloat162*>(&y);
    const uint32_t bias_bits = 0x43084308u;
    v = __hsub2(v, *reinterpret_cast<const __nv_bfloat162*>(&bias_bits));
    return *reinterpret_cast<uint32_t*>(&v);
}

// 32 consecutive 32-bit columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

}  // namespace pf

template <int N, bool TWO, bool PRE = false>
__global__ void __launch_bounds__(kPThreads, 1)
prefill_kernel(const PrefillParams p, const __grid_constant__ CUtensorMap tmV,
               const __grid_constant__ CUtensorMap tmM, const __grid_constant__ CUtensorMap tmX,
               const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2)
{
    using namespace pf;
    using Cfg = PfCfg<N, TWO, PRE>;
    // The dense-only launch lets the launches behind it start at once (programmatic dependent launch): the
    // main launch's sparse stages do not need T', and it waits (griddepcontrol.wait) just before its first
    // request of a T' tile.
    if (PRE) asm volatile("griddepcontrol.launch_dependents;");
    constexpr int kBTile = Cfg::kBTile, kStageBytes = Cfg::kStageBytes, kECol = Cfg::kECol, kPStages = Cfg::kStages;
    constexpr int kPkSlots = Cfg::kPkSlots, kDK = Cfg::kDK;
    extern __shared__ unsigned char smem_raw[];
    // layout: stages {B | A} | packed slots {value bytes | index bytes} | barriers
    unsigned char* stages = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char* packed = stages + (size_t)kPStages * kStageBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(packed + kPkSlots * kPkSlotBytes);
    uint64_t* b_full = bars;                         // [kPStages] token tile (and A2 tile) landed
    uint64_t* conv_done = bars + kPStages;           // [kPStages]
    uint64_t* empty = bars + 2 * kPStages;           // [kPStages]
    uint64_t* pk_full = bars + 3 * kPStages;         // [kPkSlots]
    uint64_t* pk_empty = pk_full + kPkSlots;         // [kPkSlots]
    uint64_t* acc_full = pk_empty + kPkSlots;        // [1]
    uint64_t* peer_ready = acc_full + 1;             // [kPStages] pair only: the odd CTA's stage is ready
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(peer_ready + kPStages);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = TWO ? cluster_rank() : 0u;           // 0 = the CTA that issues the pair's MMAs
    const int m0 = blockIdx.x * kPM, n0 = blockIdx.y * N;
    const int nb0 = n0 + (int)rank * Cfg::kBRows;                // first token row this CTA loads
    const int k_first = PRE && p.part ? (int)blockIdx.z * p.k_per : 0;      // first dense stage of this K slice
    const int n_total = PRE && p.part ? min(p.k_per, p.n2 - k_first) : p.n1 + p.n2;
    // CTAs that share token rows start their walk over the weight columns at different places,
    // so that at any moment they ask the L2 for different lines of X rather than all for the same
    // ones.  The walk is rotated by whole 256-column groups (a pair of CTAs rotates together).
    const int n_groups = ceil_div(p.n1, kPkStages);
    const int rot_g = (p.n1 % kPkStages == 0 && n_groups > 0)
                          ? (int)(((blockIdx.x >> (TWO ? 1 : 0)) + 3u * blockIdx.y) % (unsigned)n_groups) : 0;

    if (threadIdx.x == 0) PSTAMP(5, 44);
    if (threadIdx.x == 0) {
        for (int i = 0; i < kPStages; ++i) {
            mbar_init(&b_full[i], 1);
            mbar_init(&conv_done[i], TWO ? kConvWarps : kConvWarps / 2); mbar_init(&empty[i], 1); mbar_init(&peer_ready[i], 1);
        }
        for (int i = 0; i < kPkSlots; ++i) { mbar_init(&pk_full[i], 1); mbar_init(&pk_empty[i], kConvWarps); }
        mbar_init(acc_full, 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (TWO) cluster_sync_all();                    // both CTAs' barriers exist before anything crosses
    if (warp == kWarpMma) {
        if (TWO) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(s32(tmem_slot)), "r"(Cfg::kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(s32(tmem_slot)), "r"(Cfg::kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_slot);
    bool ok = true;
    if (threadIdx.x == 0) PSTAMP(5, 45);

    if (warp == kWarpXEven || warp == kWarpXOdd) {
        // ============================ token-tile producers ============================
        // Each of the two warps walks every second stage in order (a waiter that skipped uses of
        // a barrier would mistake an old phase for the one it needs).  Sparse stage: lane 0
        // requests the token tile.  Dense stage: lanes 0 and 1 request the token tile and the A2
        // tile with one instruction.
        bool t_ready = PRE;                                 // main launch: T' (and everything before it) is complete
        for (int it = warp == kWarpXEven ? 0 : 1; it < n_total; it += 2) {
            const int st = it % kPStages;
            const bool sparse = it < p.n1;
            if (!sparse && !t_ready) {
                asm volatile("griddepcontrol.wait;" ::: "memory");
                asm volatile("fence.proxy.async;" ::: "memory");   // the tiles are read by the async proxy
                t_ready = true;
            }
            // The whole warp waits (no lane is left behind at a warp barrier while another
            // spins: that costs some hundred nanoseconds per stage); lane 0 arms the barrier.
            if (it >= kPStages) ok = mbar_wait(&empty[st], ((it / kPStages) & 1) ^ 1, abort_flag) && ok;
            // dense stage: kDK columns of the token rows and of the A2 rows
            if (lane == 0) mbar_expect_tx(&b_full[st], (uint32_t)(sparse ? kBTile : (Cfg::kBRows + kPM) * kDK * 2));
            unsigned char* sbase = stages + (size_t)st * kStageBytes;
            int kb = sparse ? it + rot_g * kPkStages : it - p.n1 + k_first;
            if (sparse && kb >= p.n1) kb -= p.n1;
            const int k = sparse ? kb * kPBK : kb * kDK;
            // lane 0: the token tile (one box); lane 1, dense stages only: the A2 tile
            if (lane == 0 || (lane == 1 && !sparse))
                tma_tile(lane == 0 ? sbase : sbase + kBTile, lane == 1 ? &tmA2 : (sparse ? &tmX : &tmB2), k,
                         lane == 0 ? nb0 : m0, &b_full[st]);
            if (lane == 0) PSTAMP(0, it);
        }
    } else if (warp == kWarpPk) {
        // ============================ packed-tile producer ============================
        // lanes 0 and 1 request the value-byte and the index-byte tile with one instruction
        for (int gi = 0; gi < n_groups; ++gi) {
            const int slot = gi % kPkSlots;
            const int g = gi + rot_g < n_groups ? gi + rot_g : gi + rot_g - n_groups;
            if (gi >= kPkSlots) ok = mbar_wait(&pk_empty[slot], ((gi / kPkSlots) & 1) ^ 1, abort_flag) && ok;
            if (lane == 0) mbar_expect_tx(&pk_full[slot], (uint32_t)kPkSlotBytes);
            unsigned char* dst = packed + slot * kPkSlotBytes + (lane == 0 ? 0 : kValsTile);
            if (lane < 2) tma_tile(dst, lane == 0 ? &tmV : &tmM, g * (lane == 0 ? 64 : 32), m0, &pk_full[slot]);
        }
    } else if (warp == kWarpMma) {
        // ============================ MMA issuer ============================
        // One elected lane walks the stages and issues.
        if (TWO && rank != 0) {
            // Odd CTA of a pair: tell the even CTA when this CTA's token rows (and A2 rows) of a
            // stage have landed.  The data stay in this CTA's shared memory and are read by this
            // SM's tensor core, so an arrival ordered after the landing within this CTA is enough;
            // a cluster-scope release costs some 300 cycles per stage.
            if (lane == 0) {
                for (int it = 0; it < n_total; ++it) {
                    const int st = it % kPStages;
                    ok = mbar_wait(&b_full[st], (it / kPStages) & 1, abort_flag) && ok;
                    mbar_arrive_remote(peer_addr(&peer_ready[st], 0));
                    PSTAMP(5, it);
                }
            }
        } else if (elect_one()) {
            constexpr uint32_t idesc = idesc_bf16(TWO ? 2 * kPM : kPM, N);
            uint32_t pre = 0;       // the coming stage was found ready by an early test
            for (int it = 0; it < n_total; ++it) {
                const int st = it % kPStages;
                const uint32_t parity = (it / kPStages) & 1;
                const bool sparse = it < p.n1;
                // token tile landed; converters done (in a pair: both CTAs', reported here); the other CTA's loads landed
                if (!pre)
                    ok = mbar_wait_all(&b_full[st], parity, false, sparse ? &conv_done[st] : nullptr, parity, TWO,
                                       TWO ? &peer_ready[st] : nullptr, parity, true, abort_flag) && ok;
                fence_after_sync();
                // ask about the next stage now, without waiting: the answer comes back while this stage's
                // MMAs are issued, and in steady state it is yes
                pre = 0;
                if (it + 1 < n_total) {
                    const int st1 = (it + 1) % kPStages;
                    const uint32_t par1 = ((it + 1) / kPStages) & 1;
                    pre = mbar_test(&b_full[st1], par1, false);
                    if (it + 1 < p.n1) pre &= mbar_test(&conv_done[st1], par1, TWO);
                    if (TWO) pre &= mbar_test(&peer_ready[st1], par1, true);
                }
                const uint32_t b_addr = s32(stages + (size_t)st * kStageBytes);
                const uint32_t a_addr = b_addr + kBTile;
                PSTAMP(3, it);
                if (sparse) {
                    // per MMA: A 16 stored bf16 (32 bytes of a 64-byte row), B 32 columns (64 bytes)
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const uint32_t acc = (it > 0 || j > 0) ? 1u : 0u;
                        if (TWO) mma_sparse2(tmem_base, smem_desc64(a_addr + 32 * j), smem_desc(b_addr + 64 * j),
                                             tmem_base + kECol + 4 * st, idesc | (1u << 2) | (uint32_t)j, acc);
                        else     mma_sparse(tmem_base, smem_desc64(a_addr + 32 * j), smem_desc(b_addr + 64 * j),
                                            tmem_base + kECol + 4 * st, idesc | (1u << 2) | (uint32_t)j, acc);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < kDK / 16; ++j) {
                        const uint32_t acc = (it > 0 || j > 0) ? 1u : 0u;
                        // 32-column stages: 64-byte rows with the 64-byte swizzle; 64-column stages: 128-byte rows
                        if (TWO)            mma_dense2(tmem_base, smem_desc64(a_addr + 32 * j), smem_desc64(b_addr + 32 * j), idesc, acc);
                        else if (kDK == 32) mma_dense(tmem_base, smem_desc64(a_addr + 32 * j), smem_desc64(b_addr + 32 * j), idesc, acc);
                        else                mma_dense(tmem_base, smem_desc(a_addr + 32 * j), smem_desc(b_addr + 32 * j), idesc, acc);
                    }
                }
                // the stage is free (in both CTAs of a pair) once these MMAs have read it
                if (TWO) { mma_commit2(peer_addr(&empty[st], 0)); mma_commit2(peer_addr(&empty[st], 1)); }
                else mma_commit(&empty[st]);
                PSTAMP(4, it);
            }
            if (TWO) { mma_commit2(peer_addr(acc_full, 0)); mma_commit2(peer_addr(acc_full, 1)); }
            else mma_commit(acc_full);
        }
    } else {
        // ============================ converters, then epilogue ============================
        // Two groups of four warps take every second stage each, so that the latency chain of one
        // stage (load, expand, store, index words into TMEM, fences, arrival) overlaps the next
        // stage's.  Within a group a thread owns one weight row of the tile.
        const int row = threadIdx.x & 127;           // weight row inside the tile = TMEM lane
        const int half = threadIdx.x >> 7;           // converter group; in the epilogue, which half of the columns
        const int x = (row >> 3) & 1;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        for (int it = half; it < p.n1; it += 2) {
            const int st = it % kPStages;
            const int gi = it / kPkStages, q = it % kPkStages, slot = gi % kPkSlots;
            const unsigned char* pk = packed + slot * kPkSlotBytes;
            // the packed tile has landed, and the MMAs of the previous use of this stage are done with
            // its A tile and index words
            ok = mbar_wait_all(&pk_full[slot], (gi / kPkSlots) & 1, false, it >= kPStages ? &empty[st] : nullptr,
                               ((it / kPStages) & 1) ^ 1, false, nullptr, 0, false, abort_flag) && ok;
            if ((threadIdx.x & 127) == 0) PSTAMP(1, it);
            // ---- 16 value bytes -> 32 bf16: the row's four 16-byte chunks (64-byte rows, 64-byte swizzle)
            // the packed tiles are stored with the 64-byte (values) and 32-byte (indices) TMA swizzles so
            // that a warp's row-strided reads spread over the banks
            const uint4 v = *reinterpret_cast<const uint4*>(pk + row * 64 + (((q ^ (row >> 1)) & 3) << 4));
            const uint2 mw2 = *reinterpret_cast<const uint2*>(pk + kValsTile + row * 32 + ((((q >> 1) ^ (row >> 2)) & 1) << 4) + (q & 1) * 8);
            unsigned char* arow = stages + (size_t)st * kStageBytes + kBTile + row * 64;
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t ws = w[c] >> 4;
                uint4 o;
                o.x = nib2bf16<0>(w[c], ws); o.y = nib2bf16<1>(w[c], ws);
                o.z = nib2bf16<2>(w[c], ws); o.w = nib2bf16<3>(w[c], ws);
                *reinterpret_cast<uint4*>(arow + (((c ^ (row >> 1)) & 3) << 4)) = o;
            }
            // ---- index words of the stage's two MMAs (layout in the file header)
            uint32_t e[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const uint32_t mw = h ? mw2.y : mw2.x;
                const uint32_t send = x ? (mw & 0xFFFFu) : (mw >> 16);
                const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, 8);
                e[h] = x ? ((mw & 0xFFFF0000u) | recv) : ((mw & 0xFFFFu) | (recv << 16));
            }
            asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%0], {%1, %2};"
                         :: "r"(tmem_base + lane_base + kECol + 4 * st), "r"(e[0]), "r"(e[1]) : "memory");
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // A is read by the tensor core
            fence_before_sync();
            // one arrival per warp: arrivals on one barrier are served one after another
            __syncwarp();
            if (lane == 0) {
                // a pair's MMAs are issued by the even CTA: both CTAs' converters report there
                if (TWO && rank != 0) mbar_arrive_remote(peer_addr(&conv_done[st], 0));
                else mbar_arrive(&conv_done[st]);
                // this group's last stage of the packed tile
                if (q >= 2 || it + 2 >= p.n1) mbar_arrive(&pk_empty[slot]);
            }
            if ((threadIdx.x & 127) == 0) PSTAMP(2, it);
        }
        // ---- epilogue: thread = output row, TMEM columns = tokens; the two halves split the columns
        ok = mbar_wait(acc_full, 0, abort_flag) && ok;
        fence_after_sync();
        if (threadIdx.x == 0) PSTAMP(5, 46);
        const int orow = m0 + row;
#pragma unroll 1
        for (int c0 = half * (N / 2); c0 < (half + 1) * (N / 2); c0 += 32) {
            uint32_t r[32];
            tmem_ld32(tmem_base + lane_base + c0, r);
            if (orow < p.m_total) {
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const int token = n0 + c0 + c;
                    if (token < p.b) {
                        if (PRE && p.part) p.part[((size_t)blockIdx.z * p.b + token) * p.ldo + orow] = __uint_as_float(r[c]);
                        else p.out[(size_t)token * p.ldo + orow] = __float2bfloat16_rn(p.scale * __uint_as_float(r[c]));
                    }
                }
            }
        }
    }

    if (threadIdx.x == 0) PSTAMP(5, 47);
    if (!ok && lane == 0) flag_error(p.status, SLIM_ERR_TIMEOUT);
    fence_before_sync();
    __syncthreads();
    if (TWO) cluster_sync_all();                    // neither CTA leaves while the other may still read its shared memory
    if (warp == kWarpMma) {
        fence_after_sync();
        if (TWO) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(Cfg::kTmemCols) : "memory");
        else     asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(Cfg::kTmemCols) : "memory");
    }
}

// Sum of the K slices' partial tiles, scaled and rounded to bf16 (fixed order: deterministic).
__global__ void pre_reduce_kernel(const float* __restrict__ part, int slices, size_t n, float scale, __nv_bfloat16* __restrict__ out)
{
    // lets the main launch start, then waits for the dense-only launch whose partial tiles it adds
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < n; i += (size_t)gridDim.x * blockDim.x * 4) {
        float4 acc = *reinterpret_cast<const float4*>(part + i);
        for (int z = 1; z < slices; ++z) {
            const float4 v = *reinterpret_cast<const float4*>(part + (size_t)z * n + i);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        __nv_bfloat162 lo = __floats2bfloat162_rn(scale * acc.x, scale * acc.y), hi = __floats2bfloat162_rn(scale * acc.z, scale * acc.w);
        uint2 o; o.x = *reinterpret_cast<uint32_t*>(&lo); o.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(out + i) = o;
    }
}

// ------------------------------------------------------------------ host side
// Shape of the dense-only launch T' = X R^T: token tile, K slices, stages per slice.  The product
// has few tiles (r / 128 x tokens / tile), so K is split until they about fill the machine.
struct PrePlan { int n_tok; int slices; int k_per; };
// `overlapped`: the main launch has sparse stages to run meanwhile.  A short product with few tiles is then
// better left whole on few SMs -- no partial tiles, no reduction, and the other SMs go to the main launch at
// once -- than split over the machine (measured: 4096 columns and 32 tiles gain 2-6 %; longer or wider
// products lose, their T' arrives after the main launch's first CTAs want it).
static PrePlan pre_plan(int b, int d_in, int r, int sm_count, bool overlapped = false) {
    PrePlan pl;
    pl.n_tok = b >= 192 ? 256 : 64;
    const int tiles = ceil_div(r, kPM) * ceil_div(b, pl.n_tok);
    const int n2 = d_in / kPBK;
    int ks = overlapped && n2 <= 64 && tiles <= sm_count / 4 ? 1 : sm_count / (tiles > 0 ? tiles : 1);
    ks = ks < 1 ? 1 : (ks > 8 ? 8 : ks);
    if (ks > n2) ks = n2 > 0 ? n2 : 1;
    pl.k_per = ceil_div(n2, ks);
    pl.slices = ceil_div(n2, pl.k_per);          // every slice has at least one stage
    return pl;
}
static int pre_sm_count() {
    slim_status_t err = SLIM_OK;
    const DeviceInfo* di = device_info(&err);
    return di && di->sm_count > 0 ? di->sm_count : 148;
}

typedef CUresult (*PfEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Row-major 2-D tensor [rows][row_elems]; box of box_rows x box_elems elements.
static bool pf_map(CUtensorMap* map, const void* base, CUtensorMapDataType type, int esize, uint64_t row_elems,
                   uint64_t rows, int box_elems, int box_rows, int swizzle_bytes) {
    PfEncodeTiledFn fn = reinterpret_cast<PfEncodeTiledFn>(tensor_map_encoder());
    if (!fn) return false;
    cuuint64_t dims[2] = {row_elems, rows};
    cuuint64_t strides[1] = {row_elems * (uint64_t)esize};
    cuuint32_t box[2] = {(cuuint32_t)box_elems, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, type, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool prefill_supports(int b, int d_out, int d_in, int r) {
    // d_in % 128: the rows of the index-byte array (d_in / 8 bytes) must be a multiple of 16 bytes for TMA
    return b >= 1 && d_out % kPM == 0 && d_in % 128 == 0 && r % 16 == 0 && r >= 0;
}

size_t prefill_workspace_bytes(int b, int d_out, int d_in, int r) {
    if (!prefill_supports(b, d_out, d_in, r)) return 0;
    const size_t tq = ((size_t)b * (size_t)r * sizeof(__nv_bfloat16) + 255) / 256 * 256;
    if (r == 0) return tq;
    const PrePlan pl = pre_plan(b, d_in, r, pre_sm_count());
    return tq + (pl.slices > 1 ? (size_t)pl.slices * b * r * sizeof(float) : 0);
}

static std::atomic<bool> g_prefill_attr_set[64];   // attributes set once per device (setting them twice is harmless)

template <int N, bool TWO, bool PRE = false>
static slim_status_t launch_tile_kernel(const PrefillParams& q, int m_rows, const CUtensorMap& tmV, const CUtensorMap& tmM,
                                        const CUtensorMap& tmX, const CUtensorMap& tmA2, const CUtensorMap& tmB2,
                                        cudaStream_t st, int slices = 1, bool after_dense_only = false) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ceil_div(m_rows, kPM), ceil_div(q.b, N), slices);
    cfg.blockDim = dim3(kPThreads);
    cfg.dynamicSmemBytes = PfCfg<N, TWO, PRE>::kSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = TWO ? 2 : 1; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    // may start while the launch before it (the dense-only launch or its reduction) still runs
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = after_dense_only ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, prefill_kernel<N, TWO, PRE>, q, tmV, tmM, tmX, tmA2, tmB2);
    count_launch(1);
    return e == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

slim_status_t launch_prefill(const __nv_bfloat16* X, int b, const uint8_t* vals, const uint8_t* meta,
                             float s, const __nv_bfloat16* L, const __nv_bfloat16* R, int r,
                             int d_out, int d_in, __nv_bfloat16* Y, void* ws, uint32_t* status_dev,
                             cudaStream_t st, bool force_pair)
{
    slim_status_t err;
    const DeviceInfo* di = device_info(&err);
    if (!di) return err;
    if (!prefill_supports(b, d_out, d_in, r)) return SLIM_ERR_UNSUPPORTED_SHAPE;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !g_prefill_attr_set[dev].load(std::memory_order_acquire)) {
        if (cudaFuncSetAttribute(prefill_kernel<256, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PfCfg<256, true>::kSmem) != cudaSuccess ||
            cudaFuncSetAttribute(prefill_kernel<256, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PfCfg<256, false>::kSmem) != cudaSuccess ||
            cudaFuncSetAttribute(prefill_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PfCfg<64, false>::kSmem) != cudaSuccess ||
            cudaFuncSetAttribute(prefill_kernel<64, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PfCfg<64, false, true>::kSmem) != cudaSuccess ||
            cudaFuncSetAttribute(prefill_kernel<256, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PfCfg<256, false, true>::kSmem) != cudaSuccess)
            return SLIM_ERR_CUDA;
        g_prefill_attr_set[dev].store(true, std::memory_order_release);
    }
    __nv_bfloat16* Tq = reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<char*>(ws) + SLIM_WORKSPACE_SYNC_BYTES);
    const float s_eff = s != 0.f ? s : 1.f;       // with s == 0 only the adapter term remains
    // token tile: 256 when that gives a quarter of the SMs or more a tile, else 64 (measured: with 64 tiles of
    // 128 x 256 on 148 SMs the wide variant is a third faster than 256 tiles of 128 x 64; with 32 it is slower)
    const bool wide = force_pair || (long long)(d_out / kPM) * ceil_div(b, 256) * 4 >= (long long)di->sm_count;
    const int n_pre = 64;                         // the T' product has few row tiles: narrow token tiles fill the machine
    // The CTA-pair kernel (prefill_kernel<256, true>) measures 3-8 % faster than one CTA per tile on
    // problems with adapters and a thousand tiles or more (the 70B layers at 4096 tokens) and the same or
    // a little slower below that: it runs for those, or when asked for by name.
    if (force_pair && (d_out / kPM) % 2 != 0) return SLIM_ERR_UNSUPPORTED_SHAPE;
    const bool pair = force_pair || (wide && r > 0 && (d_out / kPM) % 2 == 0 &&
                                     (long long)(d_out / kPM) * ceil_div(b, 256) >= 1024);
    const int xbox = wide ? (pair ? 128 : 256) : 64;      // token rows one CTA loads per stage = one TMA box
    const int dk = PfCfg<256, false>::kDK;                // columns of a dense stage of the main kernels
    CUtensorMap tmV, tmM, tmX, tmXpre, tmA2, tmB2;
    bool ok = pf_map(&tmV, vals, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)d_in / 4, (uint64_t)d_out, kPkStages * kPBK / 4, kPM, 64) &&
              pf_map(&tmM, meta, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)d_in / 8, (uint64_t)d_out, kPkStages * kPBK / 8, kPM, 32) &&
              pf_map(&tmX, X, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)d_in, (uint64_t)b, 64, xbox, 128);
    if (!ok) return SLIM_ERR_CUDA;
    if (r > 0) {
        // T' = (X R^T) / s : dense phase only, output rows = adapter index
        const PrePlan pl = pre_plan(b, d_in, r, di->sm_count, s != 0.f);
        ok = pf_map(&tmA2, R, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)d_in, (uint64_t)r, 64, kPM, 128) &&
             pf_map(&tmXpre, X, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)d_in, (uint64_t)b, 64, pl.n_tok, 128);
        if (!ok) return SLIM_ERR_CUDA;
        PrefillParams q;
        q.out = Tq; q.ldo = r; q.m_total = r; q.b = b; q.n1 = 0; q.n2 = d_in / kPBK; q.scale = 1.f / s_eff; q.status = status_dev;
        q.k_per = pl.k_per;
        // partial tiles of the K slices follow T' in the workspace
        q.part = pl.slices > 1 ? reinterpret_cast<float*>(reinterpret_cast<char*>(Tq) + ((size_t)b * r * sizeof(__nv_bfloat16) + 255) / 256 * 256) : nullptr;
        slim_status_t rc = pl.n_tok == 256 ? launch_tile_kernel<256, false, true>(q, r, tmV, tmM, tmXpre, tmA2, tmXpre, st, pl.slices)
                                           : launch_tile_kernel<64, false, true>(q, r, tmV, tmM, tmXpre, tmA2, tmXpre, st, pl.slices);
        if (rc != SLIM_OK) return rc;
        if (q.part) {
            const size_t n = (size_t)b * r;
            // a small grid: its blocks wait beside the dense-only launch's and must leave room for the main launch's
            cudaLaunchConfig_t rc_cfg = {};
            const unsigned want = (unsigned)((n / 4 + 255) / 256), cap = (unsigned)(2 * di->sm_count);
            rc_cfg.gridDim = dim3(want < cap ? want : cap); rc_cfg.blockDim = dim3(256); rc_cfg.dynamicSmemBytes = 0; rc_cfg.stream = st;
            cudaLaunchAttribute rc_attr[1];
            rc_attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            rc_attr[0].val.programmaticStreamSerializationAllowed = 1;
            rc_cfg.attrs = rc_attr; rc_cfg.numAttrs = 1;
            const cudaError_t re = cudaLaunchKernelEx(&rc_cfg, pre_reduce_kernel, (const float*)q.part, pl.slices, n, q.scale, Tq);
            count_launch(1);
            if (re != cudaSuccess) return SLIM_ERR_CUDA;
        }
        // dense stages of the main kernel: 64 columns (128-byte rows), or 32 (64-byte rows) in the pair kernel
        ok = pf_map(&tmA2, L, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)r, (uint64_t)d_out, dk, kPM, dk == 64 ? 128 : 64) &&
             pf_map(&tmB2, Tq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)r, (uint64_t)b, dk, xbox, dk == 64 ? 128 : 64);
        if (!ok) return SLIM_ERR_CUDA;
    } else {
        tmA2 = tmX; tmB2 = tmX;       // never used when r == 0
    }
    PrefillParams p;
    p.out = Y; p.ldo = d_out; p.m_total = d_out; p.b = b;
    p.n1 = s != 0.f ? d_in / kPBK : 0;
    p.n2 = r > 0 ? ceil_div(r, dk) : 0;
    p.scale = s_eff; p.status = status_dev; p.part = nullptr; p.k_per = 0;
    if (p.n1 + p.n2 == 0)             // s == 0 and no adapters: the result is zero
        return cudaMemsetAsync(Y, 0, (size_t)b * d_out * 2, st) == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
    note_token_tile(wide ? 256 : 64);
    slim_status_t rc;
    const bool dep = r > 0 && p.n1 > 0;               // sparse stages to run while T' is being made
    if (!wide) rc = launch_tile_kernel<64, false>(p, d_out, tmV, tmM, tmX, tmA2, tmB2, st, 1, dep);
    else rc = pair ? launch_tile_kernel<256, true>(p, d_out, tmV, tmM, tmX, tmA2, tmB2, st, 1, dep)
                   : launch_tile_kernel<256, false>(p, d_out, tmV, tmM, tmX, tmA2, tmB2, st, 1, dep);
    if (rc != SLIM_OK) return rc;
    // T' and the partial tiles were written where the decode kernels keep their hand-over slots
    // (all ones = empty): leave the region as they expect it.
    if (r > 0 && cudaMemsetAsync(Tq, 0xFF, prefill_workspace_bytes(b, d_out, d_in, r), st) != cudaSuccess) return SLIM_ERR_CUDA;
    return SLIM_OK;
}

}  // namespace slim

#ifdef SLIM_PREFILL_TRACE
extern "C" int slim_debug_read_ptrace(unsigned long long* out) {
    return (int)cudaMemcpyFromSymbol(out, slim::g_ptrace, sizeof(slim::g_ptrace));
}
#endif
