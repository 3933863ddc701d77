// Decode-phase forward (b <= 16) on the decode-tiled weight: one persistent cooperative kernel
// that streams the weight and the adapters from HBM exactly once.
//
// Slots.  The three operands are cut into slots of 6 KB, each fetched by ONE copy request (on B200 a
// request costs about 300 ns of issue time whatever its size, and one instruction can start eight of
// them side by side, so a CTA needs requests of several kilobytes to keep up with its share of HBM):
//   weight slot   one 256-column block of a group of four row tiles of the tiled buffer (64 rows x 256
//                 columns, contiguous there), fetched with cp.async.bulk;
//   adapter slot  48 rows x 64 columns of R or of L (three 16-row tiles), one TMA box.
// Lists.  All slots of R, then of the weight, then of L form lists that are divided evenly, in list
// order, among all consumer warps of the grid.  A consumer warp owns a ring of slots in shared memory
// and walks its share of each list front to back, with the accumulators of the rows it is walking in
// registers; whenever its range leaves a group of rows it writes the partial tiles (fp32, MMA fragment
// order) to its slots of the workspace.  Nothing is summed across warps in shared memory, and no
// barrier is shared between consumer warps.  One producer warp requests the slots: lane w serves
// consumer warp w and requests that warp's next slot as soon as its ring has room (full / empty
// mbarrier pair per ring slot), so that the held requests do not sit in the warps that compute.
//
// Tensor-core mapping: the batch is the N dimension (one or two n-tiles of 8 tokens) of
// mma.sp::ordered_metadata.m16n8k32 for the weight (the tiled buffer holds the A registers and the
// metadata words as the instruction takes them) and of mma.m16n8k16 for the adapters.  Activations
// (and later T) sit in shared memory in B-fragment order, b tokens only.
//
// Large d_in: the activation slice a CTA can hold is bounded, so d_in is cut into KS slices and a CTA
// belongs to one slice for the R and weight phases (the L phase has no such limit).
//
// Hand-over between CTAs, without fences or grid barriers (the launch is cooperative, all CTAs are
// resident): a partial-sum slot holds a reserved NaN pattern while empty; its one reader polls it,
// takes the value and marks it empty again.
//   T = X R^T:   service warps (three per CTA) sum the partials of a 16-column piece in list order,
//                round to bf16 and publish {two columns, call number} as one 64-bit word; the call
//                number comes from a counter every CTA increments when it leaves.  The same warps then
//                bring all of T into shared memory while the weight phase runs, and arrive on a barrier
//                the consumers wait on before L.
//   Y:           the warp that holds the first L slot of a group of rows finishes those output tiles
//                when it leaves them:  Y = s * sum(weight partials) + sum(adapter partials), in list
//                order (without adapters: a last pass over the tiles).
// All polls are bounded; an expired one sets SLIM_ERR_TIMEOUT and the kernel runs on.
// Reductions have a fixed order: results are bit-identical from run to run.
#include <cuda.h>
#include <cstdlib>
#include <cstring>
#include "decode_tile.cuh"

namespace slim {

namespace {

using namespace dt;

constexpr int kCW = 8;                                  // consumer warps
constexpr int kProducerWarp = kCW;                      // one warp requests every slot of the CTA
constexpr int kSW = 3;                                  // service warps
constexpr int kThreads = (kCW + 1 + kSW) * 32;
constexpr int kWT = 4;                                  // row tiles of a weight slot (a group of the tiled layout)
constexpr int kAT = 3;                                  // row tiles of an adapter slot (48 rows)
constexpr int kACols = 64;                              // columns of an adapter slot (two steps of 32)
constexpr int kSlotBytes = 6144;
constexpr int kBlockBytes = 1536;                       // one 16-row x 256-column piece of the tiled weight
constexpr int kMaxRing = 8;                             // slots per warp
constexpr int kMaxRank = 3072;
constexpr int kMaxKS = 64;                              // k-slices the shared-memory tables hold
constexpr size_t kSmemBudget = 227 * 1024;
constexpr uint32_t kPollLimit = 1u << 20;
constexpr uint32_t kPollPause = 400;                    // ns between two polls of a slot: waiting warps must not flood the L2
constexpr unsigned long long kWaitNs = 250ull * 1000 * 1000;   // longest wait on a shared-memory barrier
constexpr uint32_t kIdleLimit = 1u << 21;               // rounds of 64 ns in which the producer warp found nothing to request
constexpr uint32_t kEmpty = 0xFFFFFFFFu;                // "no value yet" in a partial-sum slot
constexpr uint32_t kNanBits = 0x7FFFFFFFu;              // what a computed all-ones NaN is stored as
constexpr size_t kTfinalBytes = kDecodeTfinalBytes;
static_assert(16 * (size_t)(kMaxRank / 2) * 8 <= kTfinalBytes, "published T does not fit its region");

struct Params {
    const __nv_bfloat16* X; const uint8_t* W; __nv_bfloat16* Y;
    uint32_t* Ppart; uint32_t* Apart; uint32_t* Tpart;
    unsigned long long* Tfinal;          // [b][r / 2]  {bf16 pair, call number}
    unsigned long long* departures;      // CTAs that ever left a call on this workspace
    uint32_t* status;
    float s;
    int b, r, d_out, d_in;
    int KS, G;                           // k-slices; CTAs per slice
    int nblk;                            // 256-column blocks of a row
    int tilesW, tilesR;                  // d_out / 16; r / 16
    int unitsW, unitsR, unitsL;          // groups of kWT weight tiles; of kAT tiles of R; of kAT tiles of L
    int nqL;                             // adapter slots along r: ceil(r / 64)
    int wnR;                             // workers per slice in the R phase (<= G * kCW)
    int muW, muR, muL;                   // partial slots a worker owns in each phase
    int ring;                            // ring slots per warp
    int x_bytes;                         // activation slice region
};

// Optional timeline: built with -DSLIM_TILED_TRACE, lane 0 of consumer warp 0 (entries 0-7) and of service
// warp 0 (entries 8-9) of every CTA record the global timer (read back with slim_debug_read_tiled_trace).
#ifdef SLIM_TILED_TRACE
__device__ unsigned long long g_tiled_trace[256 * 16];
#define TSTAMP(w, i) do { if (warp == (w) && lane == 0) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); g_tiled_trace[blockIdx.x * 16 + (i)] = t_; } } while (0)
#else
#define TSTAMP(w, i) do { } while (0)
#endif

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Waits for a phase of a shared-memory barrier, for kWaitNs at most (a try may itself suspend the thread for
// a while, so the bound is on time and not on tries); false when it gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_u32(bar);
    unsigned long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if ((it & 63u) == 63u) {
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitNs) return false;
        }
    }
}
__device__ __forceinline__ void tma_tile(uint32_t dst, const CUtensorMap* tmap, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 :: "r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
// Contiguous bytes global -> shared (both 16-byte aligned, size a multiple of 16).
__device__ __forceinline__ void bulk_copy(uint32_t dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(dst), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// Device-scope accesses that bypass L1: the hand-over slots.
__device__ __forceinline__ uint32_t ld_gpu(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_gpu(uint32_t* p, uint32_t v) {
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_gpu64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_gpu64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" :: "l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint4 ld_gpu_v4(const uint32_t* p) {
    uint4 v;
    asm volatile("ld.relaxed.gpu.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_gpu_v4(uint32_t* p, uint4 v) {
    asm volatile("st.relaxed.gpu.global.v4.u32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint32_t slot_bits(float v) {    // fp32 bits that never equal kEmpty
    const uint32_t u = __float_as_uint(v);
    return u == kEmpty ? kNanBits : u;
}

// ---------------------------------------------------------------- even division of a list
// S list positions among Wn workers, in order: the first S % Wn workers get one more.
struct Split { int len, rem; };
__host__ __device__ __forceinline__ Split make_split(int S, int Wn) { Split sp; sp.len = S / Wn; sp.rem = S % Wn; return sp; }
__host__ __device__ __forceinline__ int split_start(const Split& sp, int w) { return w * sp.len + (w < sp.rem ? w : sp.rem); }
__host__ __device__ __forceinline__ int split_count(const Split& sp, int w) { return sp.len + (w < sp.rem ? 1 : 0); }

// Blocks [b0, b1) of k-slice ks.
__host__ __device__ __forceinline__ void slice_blocks(int ks, int KS, int nblk, int* b0, int* b1) {
    *b0 = (int)((long long)ks * nblk / KS);
    *b1 = (int)((long long)(ks + 1) * nblk / KS);
}

// One list as its readers need it, kept in shared memory: nq slots per unit, divided among the workers as
// `len` slots each plus one more for the first `rem`; reciprocals for division by multiplication (a
// hardware integer division is a long chain of dependent instructions).
struct ListTab { int nq, len, rem, edge; float r_nq, r_len, r_len1; };
__device__ __forceinline__ ListTab make_tab(int units, int nq, int Wn) {
    ListTab t;
    const Split sp = make_split(units * nq, Wn);
    t.nq = nq; t.len = sp.len; t.rem = sp.rem; t.edge = sp.rem * (sp.len + 1);
    t.r_nq = nq > 0 ? 1.f / (float)nq : 0.f; t.r_len = sp.len > 0 ? 1.f / (float)sp.len : 0.f; t.r_len1 = 1.f / (float)(sp.len + 1);
    return t;
}
// n / d for 0 <= n < 2^22, d > 0, rd = 1 / d: the float product is off by less than one, fixed up exactly.
__device__ __forceinline__ int fdiv(int n, int d, float rd) {
    int q = __float2int_rz(__int2float_rn(n) * rd);
    const int r = n - q * d;
    if (r < 0) --q; else if (r >= d) ++q;
    return q;
}
__device__ __forceinline__ int tab_owner(const ListTab& t, int pos) {
    return pos < t.edge ? fdiv(pos, t.len + 1, t.r_len1) : t.rem + fdiv(pos - t.edge, t.len, t.r_len);
}
__device__ __forceinline__ int tab_first_unit(const ListTab& t, int w) {      // first unit the range of worker w meets
    return fdiv(w * t.len + min(w, t.rem), t.nq, t.r_nq);
}

// Walks, in list order, the partial-sum slots that the workers of one phase left for one list
// unit: every worker whose range meets the unit's positions owns `mu` slots of `stride` words,
// the unit's being number (unit - first unit of the worker's range).
struct PartWalk {
    const ListTab& t; const int mu, unit; const size_t stride; uint32_t* const base;
    int w, w_last;
    __device__ PartWalk(uint32_t* base_, const ListTab& t_, int mu_, int unit_, size_t stride_, int worker0)
        : t(t_), mu(mu_), unit(unit_), stride(stride_), base(base_ + (size_t)worker0 * mu_ * stride_) {
        w = t.nq > 0 ? tab_owner(t, unit * t.nq) : 0;
        w_last = t.nq > 0 ? tab_owner(t, unit * t.nq + t.nq - 1) : -1;
    }
    __device__ uint32_t* next() {
        if (w > w_last) return nullptr;
        uint32_t* p = base + ((size_t)w * mu + (unit - tab_first_unit(t, w))) * stride;
        ++w;
        return p;
    }
};

constexpr int kBatch = 8;        // partial slots requested together (T partials)

// Adds to sum[e] (e < E: elements lane + 32 e of a fragment-ordered tile at `off` words inside a
// slot) the next up-to-kBatch slots of the walk; empties them.  Returns false when the walk is over.
template <int E>
__device__ __forceinline__ bool take_batch(PartWalk& pw, int off, int lane, float (&sum)[E], bool* ok) {
    uint32_t* ptr[kBatch];
#pragma unroll
    for (int k = 0; k < kBatch; ++k) ptr[k] = pw.next();
    if (!ptr[0]) return false;
    uint32_t v[kBatch][E];
#pragma unroll
    for (int k = 0; k < kBatch; ++k)
#pragma unroll
        for (int e = 0; e < E; ++e) v[k][e] = ptr[k] ? ld_gpu(ptr[k] + off + e * 32 + lane) : 0u;
    for (uint32_t spins = 0;; ++spins) {
        bool all = true;
#pragma unroll
        for (int k = 0; k < kBatch; ++k)
#pragma unroll
            for (int e = 0; e < E; ++e)
                if (v[k][e] == kEmpty) { v[k][e] = ld_gpu(ptr[k] + off + e * 32 + lane); all = false; }
        if (all) break;
        if (spins > kPollLimit) { *ok = false; break; }
        __nanosleep(kPollPause);
    }
#pragma unroll
    for (int k = 0; k < kBatch; ++k)
        if (ptr[k]) {
#pragma unroll
            for (int e = 0; e < E; ++e) {
                sum[e] += __uint_as_float(v[k][e]);
                st_gpu(ptr[k] + off + e * 32 + lane, kEmpty);
            }
        }
    return ptr[kBatch - 1] != nullptr;
}

constexpr int kFinishers = kCW + kSW;      // warps of a CTA that finish output tiles once their other work is done

// Finishes the output tiles of finisher `fid` of `n_fin`: Y = s * (weight partials of every k-slice, in list
// order) + (adapter partials, in list order), rounded to bf16.  Tiles are dealt out in order; a tile's
// partials are complete once every consumer warp has walked past its rows.
template <int NT>
__device__ __forceinline__ void finish_tiles(const Params& p, const ListTab* tabW, const ListTab* tabL, int fid, int n_fin,
                                             const LaneCtx& lc, uint32_t* expired) {
    constexpr int frag = NT * 128, E = NT * 4;
    constexpr int kFB = 8;                              // partials requested together (this code runs once per call and
                                                        // comes cold from the L2: it is kept small)
    const int lane = lc.lane;
    const Split spF = make_split(p.tilesW, n_fin);
    const int f0 = split_start(spF, fid), f1 = f0 + split_count(spF, fid);
    for (int tile = f0; tile < f1; ++tile) {
        float psum[E], asum[E];
#pragma unroll
        for (int e = 0; e < E; ++e) { psum[e] = 0.f; asum[e] = 0.f; }
        const int uW = tile / kWT, mW = tile % kWT, uL = tile / kAT, mL = tile % kAT;
        // walk state: k-slice of the weight partials being walked (p.KS = the adapter partials, then the end)
        int k2 = -1, w = 0, w_last = -1;
        auto next_part = [&](bool* is_adapter) -> uint32_t* {
            while (w > w_last) {
                ++k2;
                if (k2 > p.KS || (k2 == p.KS && p.r == 0)) return nullptr;
                const ListTab& t = k2 < p.KS ? tabW[k2] : tabL[0];
                const int u = k2 < p.KS ? uW : uL;
                w = tab_owner(t, u * t.nq); w_last = tab_owner(t, u * t.nq + t.nq - 1);
            }
            uint32_t* ptr;
            if (k2 < p.KS) ptr = p.Ppart + (((size_t)(k2 * p.G * kCW + w) * p.muW + (uW - tab_first_unit(tabW[k2], w))) * kWT + mW) * frag;
            else           ptr = p.Apart + (((size_t)w * p.muL + (uL - tab_first_unit(tabL[0], w))) * kAT + mL) * frag;
            *is_adapter = k2 == p.KS;
            ++w;
            return ptr;
        };
        for (bool more = true; more;) {
            uint32_t* ptr[kFB];
            bool adapter[kFB];
#pragma unroll
            for (int k = 0; k < kFB; ++k) { adapter[k] = false; ptr[k] = more ? next_part(&adapter[k]) : nullptr; if (!ptr[k]) more = false; }
            uint4 v[kFB][NT];
#pragma unroll
            for (int k = 0; k < kFB; ++k)
#pragma unroll
                for (int h = 0; h < NT; ++h) v[k][h] = ptr[k] ? ld_gpu_v4(ptr[k] + lane * E + 4 * h) : make_uint4(0, 0, 0, 0);
            for (uint32_t spins = 0;; ++spins) {
                bool all = true;
#pragma unroll
                for (int k = 0; k < kFB; ++k)
#pragma unroll
                    for (int h = 0; h < NT; ++h)
                        if (v[k][h].x == kEmpty || v[k][h].y == kEmpty || v[k][h].z == kEmpty || v[k][h].w == kEmpty) {
                            v[k][h] = ld_gpu_v4(ptr[k] + lane * E + 4 * h); all = false;
                        }
                if (all) break;
                if (spins > kPollLimit) { *expired |= 16u; break; }
                __nanosleep(kPollPause);
            }
#pragma unroll
            for (int k = 0; k < kFB; ++k)
                if (ptr[k]) {
#pragma unroll
                    for (int h = 0; h < NT; ++h) {
                        float* dstsum = adapter[k] ? asum : psum;
                        dstsum[4 * h + 0] += __uint_as_float(v[k][h].x); dstsum[4 * h + 1] += __uint_as_float(v[k][h].y);
                        dstsum[4 * h + 2] += __uint_as_float(v[k][h].z); dstsum[4 * h + 3] += __uint_as_float(v[k][h].w);
                        st_gpu_v4(ptr[k] + lane * E + 4 * h, make_uint4(kEmpty, kEmpty, kEmpty, kEmpty));
                    }
                }
        }
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const int h = e >> 2, q = e & 3;
            const int n = tile * 16 + lc.g + 8 * (q >> 1);
            const int tok = 8 * h + 2 * lc.t + (q & 1);
            if (tok < p.b) p.Y[(size_t)tok * p.d_out + n] = __float2bfloat16_rn(fmaf(psum[e], p.s, asum[e]));
        }
    }
}

// The jobs of one consumer warp: nR slots of the R list from sR, nW of the weight list, nL of the L list.
struct Jobs { int nR, sR, nW, sW, nL, sL, total; };
struct SliceGeo { bool in_slice; int ks, grp, blk0, blk1, nqW, nqR; };

__device__ __forceinline__ SliceGeo make_geo(const Params& p, int cta) {
    SliceGeo g;
    g.in_slice = cta < p.KS * p.G;
    g.ks = g.in_slice ? cta % p.KS : 0;
    g.grp = g.in_slice ? cta / p.KS : 0;
    slice_blocks(g.ks, p.KS, p.nblk, &g.blk0, &g.blk1);
    g.nqW = g.blk1 - g.blk0;                              // weight slots per group of rows in this slice
    g.nqR = (g.blk1 - g.blk0) * (256 / kACols);           // adapter slots per group of R rows in this slice
    return g;
}
__device__ __forceinline__ Jobs make_jobs(const Params& p, const SliceGeo& g, int cta, int n_ctas, int cwarp) {
    const Split spR = make_split(p.unitsR * g.nqR, p.wnR);
    const Split spW = make_split(p.unitsW * g.nqW, p.G * kCW);
    const Split spL = make_split(p.unitsL * p.nqL, n_ctas * kCW);
    const int wi = g.grp * kCW + cwarp;                   // worker number inside the slice
    const int wl = cta * kCW + cwarp;                     // worker number in the grid
    Jobs jb;
    jb.nR = g.in_slice && wi < p.wnR ? split_count(spR, wi) : 0; jb.sR = split_start(spR, wi);
    jb.nW = g.in_slice ? split_count(spW, wi) : 0; jb.sW = split_start(spW, wi);
    jb.nL = split_count(spL, wl); jb.sL = split_start(spL, wl);
    jb.total = jb.nR + jb.nW + jb.nL;
    return jb;
}

template <int NT>
__global__ void __launch_bounds__(kThreads, 1)
decode_tiled_kernel(const Params p, const __grid_constant__ CUtensorMap tmR, const __grid_constant__ CUtensorMap tmL)
{
    constexpr int frag = NT * 128;                   // words of one 16-row partial tile
    constexpr int E = NT * 4;                        // fragment elements per lane
    extern __shared__ unsigned char smem_raw[];
    // layout (1024-byte aligned for the swizzle): rings | X slice | T | barriers
    unsigned char* rings = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char* xs = rings + (size_t)kCW * p.ring * kSlotBytes;
    unsigned char* ts = xs + p.x_bytes;
    const int t_bytes = p.nqL * 2 * p.b * 64;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(ts + t_bytes);      // [kCW][kMaxRing]
    uint64_t* empty_bar = full_bar + kCW * kMaxRing;                     // [kCW][kMaxRing]
    uint64_t* t_bar = empty_bar + kCW * kMaxRing;
    ListTab* tabW = reinterpret_cast<ListTab*>(t_bar + 1);              // [KS] weight list of every k-slice
    ListTab* tabR = tabW + kMaxKS;                                       // [KS] R list of every k-slice
    ListTab* tabL = tabR + kMaxKS;                                       // [1]  L list

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_ctas = gridDim.x, cta = blockIdx.x;
    const LaneCtx lc = make_lane_ctx(lane);
    const SliceGeo geo = make_geo(p, cta);
    const int blk0 = geo.blk0, blk1 = geo.blk1, nqW = geo.nqW, nqR = geo.nqR, ks = geo.ks;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kCW * kMaxRing; ++i) { mbar_init(&full_bar[i], 1); mbar_init(&empty_bar[i], 1); }
        mbar_init(t_bar, kSW);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int k2 = threadIdx.x; k2 < p.KS; k2 += kThreads) {
        int c0, c1;
        slice_blocks(k2, p.KS, p.nblk, &c0, &c1);
        tabW[k2] = make_tab(p.unitsW, c1 - c0, p.G * kCW);
        tabR[k2] = make_tab(p.unitsR, (c1 - c0) * (256 / kACols), p.wnR);
    }
    if (threadIdx.x == kThreads - 1) tabL[0] = make_tab(p.unitsL, p.nqL, gridDim.x * kCW);
    __syncthreads();

    // which kind of wait expired, if any: reported in bits 16-23 of the status word beside SLIM_ERR_TIMEOUT
    // (1 R slot, 2 weight slot, 4 T in shared memory, 8 L slot, 16 partials of an output tile,
    //  32 ring slot not freed, 64 partials of T, 128 published T)
    uint32_t expired = 0;
    TSTAMP(0, 0);
#ifdef SLIM_TILED_TRACE
    if (threadIdx.x == 0) { g_tiled_trace[blockIdx.x * 16 + 11] = 0; g_tiled_trace[blockIdx.x * 16 + 12] = 0; g_tiled_trace[blockIdx.x * 16 + 14] = 0; g_tiled_trace[blockIdx.x * 16 + 13] = clock64(); }
#endif
    if (warp == kProducerWarp) {
        // ================================ producer warp ================================
        // Every lane walks the job list of its consumer warp at its own pace: in each round a lane whose
        // next ring slot is free (a test that does not wait) requests its next job, the others sit the
        // round out; the requests of a round start with one instruction per list kind.
        const bool serves = lane < kCW;
        const Jobs jb = make_jobs(p, geo, cta, n_ctas, serves ? lane : 0);
        const int total = serves ? jb.total : 0;
        uint64_t* fbar = full_bar + (serves ? lane : 0) * kMaxRing;
        uint64_t* ebar = empty_bar + (serves ? lane : 0) * kMaxRing;
        const uint32_t ring0 = smem_u32(rings + (size_t)(serves ? lane : 0) * p.ring * kSlotBytes);
        // running (group of rows, slot in group) of this lane's position in each list
        int r_u = nqR > 0 ? jb.sR / nqR : 0, r_q = nqR > 0 ? jb.sR % nqR : 0;
        int w_u = jb.sW / nqW, w_q = jb.sW % nqW;
        int l_u = p.nqL > 0 ? jb.sL / p.nqL : 0, l_q = p.nqL > 0 ? jb.sL % p.nqL : 0;
        int j = 0, slot = 0;
        uint32_t parity = 0;                                // phase of the "slot left" barrier awaited in the second lap; flips per lap
        for (uint32_t idle = 0;;) {
            const bool has = j < total;
            if (!__any_sync(0xffffffffu, has)) break;
            bool can = has;
            if (has && j >= p.ring) {
                uint32_t ok_;
                asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                             : "=r"(ok_) : "r"(smem_u32(&ebar[slot])), "r"(parity) : "memory");
                can = ok_ != 0;
            }
            if (can) {
                uint64_t* bar = &fbar[slot];
                const uint32_t dst = ring0 + slot * kSlotBytes;
                if (j < jb.nR) {
                    mbar_arrive_expect_tx(bar, kSlotBytes);
                    tma_tile(dst, &tmR, blk0 * 256 + r_q * kACols, r_u * (16 * kAT), bar);
                    if (++r_q == nqR) { r_q = 0; ++r_u; }
                } else if (j < jb.nR + jb.nW) {
                    mbar_arrive_expect_tx(bar, kSlotBytes);                     // groups are whole: the last one is padded
                    bulk_copy(dst, p.W + ((size_t)w_u * p.nblk + (size_t)(blk0 + w_q)) * kSlotBytes, kSlotBytes, bar);
                    if (++w_q == nqW) { w_q = 0; ++w_u; }
                } else {
                    mbar_arrive_expect_tx(bar, kSlotBytes);
                    tma_tile(dst, &tmL, l_q * kACols, l_u * (16 * kAT), bar);
                    if (++l_q == p.nqL) { l_q = 0; ++l_u; }
                }
                if (++slot == p.ring) { slot = 0; if (j >= p.ring) parity ^= 1u; }
                ++j;
            }
            if (__any_sync(0xffffffffu, can)) idle = 0;
            else {
                if (++idle > kIdleLimit) { expired |= 32u; break; }
                __nanosleep(64);
            }
        }
    } else if (warp < kCW) {
        // ================================ consumer warps ================================
        const Jobs jb = make_jobs(p, geo, cta, n_ctas, warp);
        const int nR = jb.nR, sR = jb.sR, nW = jb.nW, sW = jb.sW, nL = jb.nL, sL = jb.sL;
        const int wi = geo.grp * kCW + warp, wl = cta * kCW + warp;
        uint64_t* my_full = full_bar + warp * kMaxRing;
        uint64_t* my_empty = empty_bar + warp * kMaxRing;
        const uint32_t my_ring = smem_u32(rings + (size_t)warp * p.ring * kSlotBytes);

        // ---- the CTA's slice of the activations into shared memory, fragment order.  A thread
        // requests several 16-byte pieces before it stores the first (one global round trip per batch).
        if (geo.in_slice) {
            const int cols = (blk1 - blk0) * 256, chunks = cols / 8;      // 16-byte chunks per token
            const __nv_bfloat16* xsrc = p.X + (size_t)blk0 * 256;
            const int n_chunks = p.b * chunks;
            constexpr int kXBatch = 8;
            for (int i0 = threadIdx.x; i0 < n_chunks; i0 += kCW * 32 * kXBatch) {
                uint4 v[kXBatch];
#pragma unroll
                for (int k = 0; k < kXBatch; ++k) {
                    const int idx = i0 + k * kCW * 32;
                    if (idx < n_chunks) {
                        const int tok = idx / chunks, c = idx - tok * chunks;
                        v[k] = __ldg(reinterpret_cast<const uint4*>(xsrc + (size_t)tok * p.d_in + 8 * c));
                    }
                }
#pragma unroll
                for (int k = 0; k < kXBatch; ++k) {
                    const int idx = i0 + k * kCW * 32;
                    if (idx < n_chunks) {
                        const int tok = idx / chunks, c = idx - tok * chunks;
                        // columns 8c .. 8c+7 = step c/4, register i = c%4, pairs t = 0..3
                        uint32_t* dst = reinterpret_cast<uint32_t*>(xs) + (((c >> 2) * p.b + tok) * 16 + (c & 3));
                        dst[0] = v[k].x; dst[4] = v[k].y; dst[8] = v[k].z; dst[12] = v[k].w;
                    }
                }
            }
        }
        asm volatile("bar.sync 1, %0;" :: "n"(kCW * 32) : "memory");          // the consumer warps only
        TSTAMP(0, 1);

        const uint32_t xs_addr = smem_u32(xs), ts_addr = smem_u32(ts);
        uint32_t* const Pmine = p.Ppart + ((size_t)(ks * p.G * kCW + wi) * p.muW) * (kWT * frag);
        uint32_t* const Tmine = p.Tpart + ((size_t)(ks * p.wnR + wi) * p.muR) * (kAT * frag);
        uint32_t* const Amine = p.Apart + ((size_t)wl * p.muL) * (kAT * frag);

        float acc[kWT][NT][4];                              // weight phase: four row tiles; adapter phases: the first three
        auto zero_acc = [&]() {
#pragma unroll
            for (int m = 0; m < kWT; ++m)
#pragma unroll
                for (int h = 0; h < NT; ++h)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[m][h][e] = 0.f;
        };
        // a partial tile in the workspace: lane-major, word lane * E + 4 h + e (every word is its own "empty" flag)
        auto store_tile = [&](uint32_t* dst, const float (&a)[NT][4]) {
#pragma unroll
            for (int h = 0; h < NT; ++h)
                st_gpu_v4(dst + lane * E + 4 * h, make_uint4(slot_bits(a[h][0]), slot_bits(a[h][1]), slot_bits(a[h][2]), slot_bits(a[h][3])));
        };

        zero_acc();
        // Walk of the three lists with running (group of rows, slot in group) pairs and a running ring
        // position: no division inside the loops (a division is a long chain of dependent instructions, and
        // a warp has only one or two others on its scheduler to hide it behind).
        int slot = 0; uint32_t parity = 0;
        auto next_slot = [&]() { if (++slot == p.ring) { slot = 0; parity ^= 1u; } };
        const int r_first = nqR > 0 ? sR / nqR : 0, w_first = sW / nqW, l_first = p.nqL > 0 ? sL / p.nqL : 0;

        // ---------------------------------------------------------------- R slots
        {
            int u = r_first, q = nqR > 0 ? sR % nqR : 0;
            for (int j = 0; j < nR; ++j) {
                const uint32_t src = my_ring + slot * kSlotBytes;
                const int mt = min(kAT, p.tilesR - u * kAT);
                if (!mbar_wait(&my_full[slot], parity)) expired |= 1u;
                if (j == 0) TSTAMP(0, 2);
#pragma unroll
                for (int jj = 0; jj < 2; ++jj) {
                    uint4 xb[NT];
                    load_x_step<NT>(xb, xs_addr, q * 2 + jj, p.b, lc);
                    if (mt == kAT) {
#pragma unroll
                        for (int m = 0; m < kAT; ++m) dense_step<NT>(acc[m], src + m * 2048, jj, xb, lc);
                    } else {
#pragma unroll
                        for (int m = 0; m < kAT; ++m)
                            if (m < mt) dense_step<NT>(acc[m], src + m * 2048, jj, xb, lc);
                    }
                }
                __syncwarp();                               // every lane is done reading the slot
                if (lane == 0) mbar_arrive(&my_empty[slot]);
                next_slot();
                if (++q == nqR || j + 1 == nR) {            // leaving the rows: their partials go to the workspace
#pragma unroll
                    for (int m = 0; m < kAT; ++m)
                        if (m < mt) store_tile(Tmine + ((size_t)(u - r_first) * kAT + m) * frag, acc[m]);
                    zero_acc();
                    q = 0; ++u;
                }
            }
        }
        // ---------------------------------------------------------------- weight slots
        {
            int u = w_first, q = sW % nqW;
            for (int j = 0; j < nW; ++j) {
                const uint32_t src = my_ring + slot * kSlotBytes;
                const int mt = min(kWT, p.tilesW - u * kWT);
#ifdef SLIM_TILED_TRACE
                const long long w0_ = clock64();
#endif
                if (!mbar_wait(&my_full[slot], parity)) expired |= 2u;
#ifdef SLIM_TILED_TRACE
                const long long c0_ = clock64();
                if (warp == 0 && lane == 0) { g_tiled_trace[blockIdx.x * 16 + 11] += c0_ - w0_; g_tiled_trace[blockIdx.x * 16 + 12] += 1; }
#endif
                if (j == 0) TSTAMP(0, 3);
                {
                    uint4 xf[8][NT];
                    load_x_block<NT>(xf, xs_addr, q * 8, p.b, lc);
                    if (mt == kWT) {                          // the usual case, free of branches between the tiles
#pragma unroll
                        for (int m = 0; m < kWT; ++m) sparse_block<NT>(acc[m], src + m * kBlockBytes, xf, lc);
                    } else {
#pragma unroll
                        for (int m = 0; m < kWT; ++m)
                            if (m < mt) sparse_block<NT>(acc[m], src + m * kBlockBytes, xf, lc);
                    }
                }
#ifdef SLIM_TILED_TRACE
                if (warp == 0 && lane == 0) g_tiled_trace[blockIdx.x * 16 + 14] += clock64() - c0_;
#endif
                __syncwarp();
                if (lane == 0) mbar_arrive(&my_empty[slot]);
                next_slot();
                if (++q == nqW || j + 1 == nW) {
#pragma unroll
                    for (int m = 0; m < kWT; ++m)
                        if (m < mt) store_tile(Pmine + ((size_t)(u - w_first) * kWT + m) * frag, acc[m]);
                    zero_acc();
                    q = 0; ++u;
                }
            }
        }
        // ---------------------------------------------------------------- L slots
        if (nL > 0) {
            TSTAMP(0, 4);
            if (!mbar_wait(t_bar, 0)) expired |= 4u;        // all of T is in shared memory
            TSTAMP(0, 5);
            int u = l_first, q = sL % p.nqL;
            for (int j = 0; j < nL; ++j) {
                const uint32_t src = my_ring + slot * kSlotBytes;
                const int mt = min(kAT, p.tilesW - u * kAT);
                if (!mbar_wait(&my_full[slot], parity)) expired |= 8u;
#pragma unroll
                for (int jj = 0; jj < 2; ++jj) {
                    uint4 tb[NT];
                    load_x_step<NT>(tb, ts_addr, q * 2 + jj, p.b, lc);
                    if (mt == kAT) {
#pragma unroll
                        for (int m = 0; m < kAT; ++m) dense_step<NT>(acc[m], src + m * 2048, jj, tb, lc);
                    } else {
#pragma unroll
                        for (int m = 0; m < kAT; ++m)
                            if (m < mt) dense_step<NT>(acc[m], src + m * 2048, jj, tb, lc);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&my_empty[slot]);
                next_slot();
                if (++q == p.nqL || j + 1 == nL) {            // leaving the rows: their partials go to the workspace
#pragma unroll
                    for (int m = 0; m < kAT; ++m)
                        if (m < mt) store_tile(Amine + ((size_t)(u - l_first) * kAT + m) * frag, acc[m]);
                    zero_acc();
                    q = 0; ++u;
                }
            }
        }
        TSTAMP(0, 6);
        finish_tiles<NT>(p, tabW, tabL, cta * kFinishers + warp, n_ctas * kFinishers, lc, &expired);
        TSTAMP(0, 7);
#ifdef SLIM_TILED_TRACE
        if (warp == 0 && lane == 0) g_tiled_trace[blockIdx.x * 16 + 13] = clock64() - g_tiled_trace[blockIdx.x * 16 + 13];
#endif
    } else {
        // ================================ service warps ================================
        const int sw = warp - kProducerWarp - 1;
        if (p.r > 0) {
        const uint32_t call = (uint32_t)(ld_gpu64(p.departures) / (unsigned)n_ctas) + 1u;
        const int pairs = p.r / 2;
        bool ok = true;
        // ---- sum the partials of T, 32 fragment elements per item, and publish them
        const int items = p.tilesR * E;
        for (int it = cta * kSW + sw; it < items; it += n_ctas * kSW) {
            const int jt = it / E, e = it % E;
            float sum[1] = {0.f};
            for (int k2 = 0; k2 < p.KS; ++k2) {
                PartWalk pw(p.Tpart, tabR[k2], p.muR, jt / kAT, (size_t)kAT * frag, k2 * p.wnR);
                while (take_batch<1>(pw, (jt % kAT) * frag + e, lane * E, sum, &ok)) { }
                if (!ok) expired |= 64u;
            }
            // element (h, q, lane) of the fragment is T[token 8h + 2(lane%4) + (q&1)][16 jt + lane/4 + 8(q>>1)]:
            // lanes 8i + t and 8i + 4 + t hold neighbouring columns
            const float other = __shfl_xor_sync(0xffffffffu, sum[0], 4);
            const int h = e >> 2, q = e & 3;
            const int tok = 8 * h + 2 * lc.t + (q & 1);
            if (!(lc.g & 1) && tok < p.b) {
                const int col = jt * 16 + lc.g + 8 * (q >> 1);
                const __nv_bfloat162 pr = __floats2bfloat162_rn(sum[0], other);
                st_gpu64(p.Tfinal + (size_t)tok * pairs + (col >> 1),
                         ((unsigned long long)call << 32) | *reinterpret_cast<const uint32_t*>(&pr));
            }
        }
        TSTAMP(kProducerWarp + 1, 8);
        // ---- all of T into shared memory (fragment order; columns past r are zero)
        const int st = threadIdx.x - (kProducerWarp + 1) * 32;
        uint32_t* tsw = reinterpret_cast<uint32_t*>(ts);
        for (int i = st; i < t_bytes / 4; i += kSW * 32) tsw[i] = 0u;
        asm volatile("bar.sync 2, %0;" :: "n"(kSW * 32) : "memory");            // the service warps only
        const int entries = p.b * pairs;
        constexpr int kFetch = 8;
        for (int e0 = st; e0 < entries; e0 += kSW * 32 * kFetch) {
            unsigned long long v[kFetch];
#pragma unroll
            for (int k = 0; k < kFetch; ++k) {
                const int e = e0 + k * kSW * 32;
                v[k] = e < entries ? ld_gpu64(p.Tfinal + e) : ((unsigned long long)call << 32);
            }
            for (uint32_t spins = 0;; ++spins) {
                bool all = true;
#pragma unroll
                for (int k = 0; k < kFetch; ++k)
                    if ((uint32_t)(v[k] >> 32) != call) { v[k] = ld_gpu64(p.Tfinal + e0 + k * kSW * 32); all = false; }
                if (all) break;
                if (spins > kPollLimit) { expired |= 128u; break; }
                __nanosleep(kPollPause);
            }
#pragma unroll
            for (int k = 0; k < kFetch; ++k) {
                const int e = e0 + k * kSW * 32;
                if (e < entries) {
                    const int tok = e / pairs, col = 2 * (e % pairs);
                    // column col = 32 step + 2 t + 8 i
                    const int step = col >> 5, i = (col >> 3) & 3, t = (col >> 1) & 3;
                    tsw[((step * p.b + tok) * 4 + t) * 4 + i] = (uint32_t)v[k];
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(t_bar);
        TSTAMP(kProducerWarp + 1, 9);
        }
        TSTAMP(kProducerWarp + 1, 10);
        finish_tiles<NT>(p, tabW, tabL, cta * kFinishers + kCW + sw, n_ctas * kFinishers, lc, &expired);
        TSTAMP(kProducerWarp + 1, 15);
    }

    if (expired && p.status) atomicOr(p.status, (1u << SLIM_ERR_TIMEOUT) | (expired << 16));
    __syncthreads();                                       // every poll of this CTA is over
    if (threadIdx.x == 0) atomicAdd(p.departures, 1ull);
}

// ------------------------------------------------------------------ host side
struct Plan {
    int nt, KS, G, nblk, ring;
    int tilesW, tilesR, unitsW, unitsR, unitsL, nqL, wnR, muW, muR, muL;
    int x_bytes;
    size_t smem, p_bytes, a_bytes, t_bytes;
};

// Slots a worker needs: one per list unit its range can meet.
int slots_per_worker(int S, int Wn, int nq) {
    if (S == 0 || nq == 0) return 1;
    const int longest = S / Wn + (S % Wn ? 1 : 0);
    return (longest + nq - 2) / nq + 1;
}

bool shape_ok(int b, int d_out, int d_in, int r) {
    return b >= 1 && b <= 16 && d_in % 256 == 0 && d_in >= 256 && d_out % 16 == 0 && d_out >= 16 && r % 16 == 0 && r >= 0 &&
           r <= kMaxRank;
}

bool make_plan(int b, int d_out, int d_in, int r, int ctas, Plan* pl) {
    if (!shape_ok(b, d_out, d_in, r) || ctas < 1) return false;
    pl->nt = b <= 8 ? 1 : 2;
    pl->nblk = d_in / 256;
    pl->tilesW = d_out / 16;
    pl->tilesR = r / 16;
    pl->unitsW = ceil_div(pl->tilesW, kWT);
    pl->unitsR = ceil_div(pl->tilesR, kAT);
    pl->unitsL = ceil_div(pl->tilesW, kAT);
    pl->nqL = ceil_div(r, kACols);
    const int workers = ctas * kCW;
    // shared memory: T, the rings, and the activation slice (b tokens x 2 bytes per column).  The rings want
    // to hold what HBM delivers during one round trip (18 KB or more per warp); the slice wants to be wide,
    // because every k-slice adds a set of partial sums.  Take the deepest ring (up to kMaxRing slots)
    // that still leaves the whole row to one slice, else three slots, else two.
    const size_t t_smem = (size_t)pl->nqL * 2 * b * 64;
    const size_t fixed = 1024 + t_smem + (2 * kCW * kMaxRing + 1) * 8 + (2 * kMaxKS + 1) * sizeof(ListTab) + 64;
    const size_t row_bytes = (size_t)pl->nblk * 512 * b;
    auto left_with = [&](int ring) -> size_t {
        const size_t used = fixed + (size_t)kCW * ring * kSlotBytes;
        return kSmemBudget > used ? kSmemBudget - used : 0;
    };
    pl->ring = 2;
    for (int ring = kMaxRing; ring >= 3; --ring)
        if (left_with(ring) >= row_bytes || (ring == 3 && left_with(3) >= (size_t)b * 512 * 4)) { pl->ring = ring; break; }
#ifdef SLIM_DECODE_TUNE
    // experiments only: the environment overrides the ring depth
    if (const char* e = getenv("SLIM_RING")) { const int v = atoi(e); if (v >= 2 && v <= kMaxRing && left_with(v) >= (size_t)b * 512) pl->ring = v; }
#endif
    const size_t left = left_with(pl->ring);
    const int max_blocks = (int)(left / ((size_t)b * 512));
    if (max_blocks < 1) return false;
    pl->KS = ceil_div(pl->nblk, max_blocks);
    if (pl->KS > ctas || pl->KS > kMaxKS) return false;
    pl->G = ctas / pl->KS;
    int widest = 0, muW = 1, muR = 1;
    const int slice_workers = pl->G * kCW;
    // R phase: eight slots or more per worker, so that a piece of T has few partials to collect (the adapter
    // arithmetic is light: a fraction of the warps keeps up with the stream, the others start on the weight)
    {
        int b0, b1;
        slice_blocks(0, pl->KS, pl->nblk, &b0, &b1);
        const int S = pl->unitsR * (b1 - b0) * (256 / kACols);
        int wn = S / 8;
        pl->wnR = wn < 1 ? 1 : (wn > slice_workers ? slice_workers : wn);
    }
    for (int ks = 0; ks < pl->KS; ++ks) {
        int b0, b1;
        slice_blocks(ks, pl->KS, pl->nblk, &b0, &b1);
        if (b1 - b0 > widest) widest = b1 - b0;
        const int nq = b1 - b0, nqr = (b1 - b0) * (256 / kACols);
        const int mw = slots_per_worker(pl->unitsW * nq, slice_workers, nq), mr = slots_per_worker(pl->unitsR * nqr, pl->wnR, nqr);
        if (mw > muW) muW = mw;
        if (mr > muR) muR = mr;
    }
    pl->muW = muW; pl->muR = muR;
    pl->muL = slots_per_worker(pl->unitsL * pl->nqL, workers, pl->nqL);
    pl->x_bytes = widest * 512 * b;
    pl->smem = fixed + (size_t)kCW * pl->ring * kSlotBytes + pl->x_bytes;
    const size_t frag_bytes = (size_t)pl->nt * 128 * sizeof(float);
    pl->p_bytes = (size_t)pl->KS * slice_workers * pl->muW * kWT * frag_bytes;
    pl->a_bytes = r > 0 ? (size_t)workers * pl->muL * kAT * frag_bytes : 0;
    pl->t_bytes = r > 0 ? (size_t)pl->KS * pl->wnR * pl->muR * kAT * frag_bytes : 0;
    return pl->smem <= kSmemBudget;
}

template <int NT>
int query_residency() {
    int n = 0;
    if (cudaFuncSetAttribute(decode_tiled_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget) != cudaSuccess)
        return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_tiled_kernel<NT>, kThreads, kSmemBudget) != cudaSuccess) return 0;
    return n > 0 ? 1 : 0;
}

int grid_ctas() {
    slim_status_t err;
    const DeviceInfo* di = device_info(&err);
    if (!di) return 148;       // sizing queries without a device assume a full B200
    return di->decode_tiled_ok ? di->sm_count : 0;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Row-major bf16 matrix [rows][cols], boxes of 48 rows x 64 columns (128-byte rows), 128-byte swizzle.
bool make_tile_map(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows) {
    EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(tensor_map_encoder());
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {kACols, 16 * kAT};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

int decode_tiled_query_residency() { return query_residency<1>() && query_residency<2>(); }

bool decode_tiled_supports(int b, int d_out, int d_in, int r) {
    Plan pl;
    const int ctas = grid_ctas();
    return ctas > 0 && make_plan(b, d_out, d_in, r, ctas, &pl);
}

size_t decode_tiled_workspace_bytes(int b, int d_out, int d_in, int r) {
    Plan pl;
    const int ctas = grid_ctas();
    if (ctas < 1 || !make_plan(b, d_out, d_in, r, ctas, &pl)) return 0;
    return kTfinalBytes + pl.p_bytes + pl.a_bytes + pl.t_bytes;
}

slim_status_t launch_decode_tiled(const __nv_bfloat16* X, int b, const uint8_t* W, float s, const __nv_bfloat16* L,
                                  const __nv_bfloat16* R, int r, int d_out, int d_in, __nv_bfloat16* Y, void* ws,
                                  uint32_t* status_dev, cudaStream_t st)
{
    slim_status_t err;
    const DeviceInfo* di = device_info(&err);
    if (!di) return err;
    Plan pl;
    const int ctas = grid_ctas();
    if (ctas < 1 || !make_plan(b, d_out, d_in, r, ctas, &pl)) return SLIM_ERR_UNSUPPORTED_SHAPE;
    Params p;
    p.X = X; p.W = W; p.Y = Y;
    char* base = reinterpret_cast<char*>(ws);
    p.departures = reinterpret_cast<unsigned long long*>(base);
    p.Tfinal = reinterpret_cast<unsigned long long*>(base + SLIM_WORKSPACE_SYNC_BYTES);
    p.Ppart = reinterpret_cast<uint32_t*>(base + SLIM_WORKSPACE_SYNC_BYTES + kTfinalBytes);
    p.Apart = reinterpret_cast<uint32_t*>(base + SLIM_WORKSPACE_SYNC_BYTES + kTfinalBytes + pl.p_bytes);
    p.Tpart = reinterpret_cast<uint32_t*>(base + SLIM_WORKSPACE_SYNC_BYTES + kTfinalBytes + pl.p_bytes + pl.a_bytes);
    p.status = status_dev;
    p.s = s; p.b = b; p.r = r; p.d_out = d_out; p.d_in = d_in;
    p.KS = pl.KS; p.G = pl.G; p.nblk = pl.nblk;
    p.tilesW = pl.tilesW; p.tilesR = pl.tilesR; p.unitsW = pl.unitsW; p.unitsR = pl.unitsR; p.unitsL = pl.unitsL;
    p.nqL = pl.nqL; p.wnR = pl.wnR; p.muW = pl.muW; p.muR = pl.muR; p.muL = pl.muL;
    p.ring = pl.ring; p.x_bytes = pl.x_bytes;
    CUtensorMap tmR, tmL;
    if (r > 0) {
        if (!make_tile_map(&tmR, R, (uint64_t)d_in, (uint64_t)r) || !make_tile_map(&tmL, L, (uint64_t)r, (uint64_t)d_out))
            return SLIM_ERR_CUDA;
    } else {
        memset(&tmR, 0, sizeof tmR); memset(&tmL, 0, sizeof tmL);      // never used when r == 0
    }
    void* args[] = {&p, &tmR, &tmL};
    const dim3 grid(ctas), block(kThreads);
    const void* fn = pl.nt == 1 ? (const void*)decode_tiled_kernel<1> : (const void*)decode_tiled_kernel<2>;
    const cudaError_t e = cudaLaunchCooperativeKernel(fn, grid, block, args, pl.smem, st);
    count_launch(1);
    return e == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

}  // namespace slim

#ifdef SLIM_TILED_TRACE
extern "C" int slim_debug_read_tiled_trace(unsigned long long* out) {
    return (int)cudaMemcpyFromSymbol(out, slim::g_tiled_trace, sizeof(slim::g_tiled_trace));
}
#endif
