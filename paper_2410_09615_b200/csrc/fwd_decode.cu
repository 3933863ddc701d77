// Decode-phase forward (b <= 16): one persistent cooperative kernel that
// streams the packed weight and the adapters from HBM exactly once.
//
// The batch is the N dimension of warp-level tensor-core MMAs (one or two
// n-tiles of 8 tokens), so the kernel stays bandwidth-bound up to b = 16:
//   * packed weight rows are the SPARSE A operand of
//     mma.sp::ordered_metadata.m16n8k32 (bf16 x bf16 -> fp32): the library's
//     value byte of one 2:4 group is exactly one thread's register pair and the
//     index nibbles are the instruction's metadata, so decoding is nibble ->
//     exact bf16 integer and nothing else;
//   * adapter rows (R in phase 1, L in phase 2) are the dense A operand of
//     mma.m16n8k16.
//
// Work split.  d_in is cut into 256-wide k-blocks; a CTA owns one k-slice of up
// to 8 blocks, one block per warp, and keeps that warp's activations as MMA B
// fragments in registers for its whole life.  CTAs are divided into weight CTAs
// and adapter (R) CTAs in proportion to the bytes each matrix streams.  A CTA
// loops over 16-row tiles of its matrix; the 8 warps' partial tiles are summed
// through shared memory and written to the workspace as split-K partials.
// After one grid-wide barrier (bounded spin on a counter; the launch is
// cooperative, so all CTAs are resident) every warp finishes 16-row output
// tiles:  Y = s * sum(partials) + T L^T  with T = sum(partials of X R^T)
// rounded once to bf16.  Reductions run in a fixed order: results are
// bit-identical from run to run.
#include "common.cuh"

namespace slim {

struct DecodeParams {
    const __nv_bfloat16* X; const uint8_t* vals; const uint8_t* meta;
    const __nv_bfloat16* L; const __nv_bfloat16* R; __nv_bfloat16* Y;
    float* Ppart; float* Tpart; uint32_t* sync; uint32_t* status;
    float s;
    int b, r, d_out, d_in;
    int KS, nblk, GW, GR, r_pad;
};

constexpr int kDecodeThreads = 256;
constexpr int kWarps = 8;
constexpr int kMaxDecodeRank = 3072;
constexpr uint32_t kSpinLimit = 1u << 22;

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
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
__device__ __forceinline__ uint32_t decode_group(uint32_t w, uint32_t w_shr4, uint32_t byte_sel) {
    uint32_t x;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(x) : "r"(w), "r"(w_shr4), "r"(byte_sel));
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

// Sum the warps' partial tiles and write one split-K partial (fragment order).
template <int NT>
__device__ __forceinline__ void reduce_and_store(float (*red)[NT * 128], const float (&acc)[NT][4],
                                                 bool active, int nb, float* dst)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (active) {
#pragma unroll
        for (int h = 0; h < NT; ++h)
#pragma unroll
            for (int q = 0; q < 4; ++q) red[warp][(h * 4 + q) * 32 + lane] = acc[h][q];
    }
    __syncthreads();
    if (threadIdx.x < NT * 128) {
        float sum = 0.f;
        for (int w = 0; w < nb; ++w) sum += red[w][threadIdx.x];
        dst[threadIdx.x] = sum;
    }
    __syncthreads();
}

template <int NT>
__global__ void __launch_bounds__(kDecodeThreads, 1)
decode_kernel(const DecodeParams p)
{
    __shared__ float red[kWarps][NT * 128];
    extern __shared__ uint4 dyn_smem[];
    __nv_bfloat16* Ts = reinterpret_cast<__nv_bfloat16*>(dyn_smem);   // [NT*8][r_pad]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int tilesW = p.d_out / 16, tilesR = p.r / 16;
    const int frag = NT * 128;

    // ------------------------------------------------------------ phase 1
    {
        const int cta = blockIdx.x;
        const int nW = p.KS * p.GW;
        const bool wrole = cta < nW;
        const int c2 = wrole ? cta : cta - nW;
        const int ks = c2 % p.KS, grp = c2 / p.KS;
        const int blk_begin = (int)((long long)ks * p.nblk / p.KS);
        const int nb = (int)((long long)(ks + 1) * p.nblk / p.KS) - blk_begin;
        const bool active = warp < nb;
        const size_t kbase = (size_t)(blk_begin + warp) * 256;

        if (wrole) {
            // activations as sparse-MMA B fragments: step j, n-tile h, register i
            // holds X[g + 8h][kbase + 32j + 2t + 8i .. +1]
            uint32_t xf[8][NT][4];
#pragma unroll
            for (int j = 0; j < 8; ++j)
#pragma unroll
                for (int h = 0; h < NT; ++h)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int row = g + 8 * h;
                        xf[j][h][i] = (active && row < p.b)
                            ? __ldg(reinterpret_cast<const uint32_t*>(p.X + (size_t)row * p.d_in + kbase + 32 * j + 2 * t + 8 * i))
                            : 0u;
                    }
            const uint32_t byte_sel = (uint32_t)t * 0x1111u + 0x4400u;   // bytes {t, t, 4+t, 4+t}
            const uint32_t meta_sel = (t & 1) ? 0x7632u : 0x5410u;
            const size_t vstride = (size_t)p.d_in / 4, mstride = (size_t)p.d_in / 8;
            for (int tile = grp; tile < tilesW; tile += p.GW) {
                float acc[NT][4];
#pragma unroll
                for (int h = 0; h < NT; ++h)
#pragma unroll
                    for (int q = 0; q < 4; ++q) acc[h][q] = 0.f;
                if (active) {
                    const size_t row0 = (size_t)tile * 16 + g, row1 = row0 + 8;
                    const uint8_t* v0p = p.vals + row0 * vstride + (kbase >> 2);
                    const uint8_t* v1p = p.vals + row1 * vstride + (kbase >> 2);
                    uint4 v0[4], v1[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) { v0[i] = ldg_stream(v0p + 16 * i); v1[i] = ldg_stream(v1p + 16 * i); }
                    // the metadata of steps 0-3 is supplied by threads 0,1 of a quad,
                    // that of steps 4-7 by threads 2,3: each loads its own 16 bytes
                    const uint4 m0 = ldg_stream(p.meta + row0 * mstride + (kbase >> 3) + 16 * (t >> 1));
                    const uint4 m1 = ldg_stream(p.meta + row1 * mstride + (kbase >> 3) + 16 * (t >> 1));
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t w0a = word_of(v0[j >> 1], (2 * j) & 3), w0b = word_of(v0[j >> 1], (2 * j + 1) & 3);
                        const uint32_t w1a = word_of(v1[j >> 1], (2 * j) & 3), w1b = word_of(v1[j >> 1], (2 * j + 1) & 3);
                        uint32_t a[4];
                        a[0] = decode_group(w0a, w0a >> 4, byte_sel);
                        a[1] = decode_group(w1a, w1a >> 4, byte_sel);
                        a[2] = decode_group(w0b, w0b >> 4, byte_sel);
                        a[3] = decode_group(w1b, w1b >> 4, byte_sel);
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
                reduce_and_store<NT>(red, acc, active, nb, p.Ppart + ((size_t)ks * tilesW + tile) * frag);
            }
        } else {
            // activations as dense-MMA B fragments: block jj (32 columns), n-tile h:
            // 16 bytes X[g + 8h][kbase + 32jj + 8t .. +8)
            uint4 xd[8][NT];
#pragma unroll
            for (int jj = 0; jj < 8; ++jj)
#pragma unroll
                for (int h = 0; h < NT; ++h) {
                    const int row = g + 8 * h;
                    xd[jj][h] = (active && row < p.b)
                        ? __ldg(reinterpret_cast<const uint4*>(p.X + (size_t)row * p.d_in + kbase + 32 * jj + 8 * t))
                        : make_uint4(0, 0, 0, 0);
                }
            for (int tile = grp; tile < tilesR; tile += p.GR) {
                float acc[NT][4];
#pragma unroll
                for (int h = 0; h < NT; ++h)
#pragma unroll
                    for (int q = 0; q < 4; ++q) acc[h][q] = 0.f;
                if (active) {
                    const __nv_bfloat16* r0 = p.R + ((size_t)tile * 16 + g) * p.d_in + kbase + 8 * t;
                    const __nv_bfloat16* r1 = r0 + (size_t)8 * p.d_in;
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint4 ra[4], rb[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            ra[i] = ldg_stream(r0 + 32 * (4 * half + i));
                            rb[i] = ldg_stream(r1 + 32 * (4 * half + i));
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int h = 0; h < NT; ++h) {
                                const uint4 xb = xd[4 * half + i][h];
                                mma_16816(acc[h], ra[i].x, rb[i].x, ra[i].y, rb[i].y, xb.x, xb.y);
                                mma_16816(acc[h], ra[i].z, rb[i].z, ra[i].w, rb[i].w, xb.z, xb.w);
                            }
                    }
                }
                reduce_and_store<NT>(red, acc, active, nb, p.Tpart + ((size_t)ks * tilesR + tile) * frag);
            }
        }
    }

    // ------------------------------------------------- grid-wide barrier
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(&p.sync[0], 1u);
        bool ok = false;
        for (uint32_t it = 0; it < kSpinLimit; ++it) {
            if (ld_acquire(&p.sync[0]) >= gridDim.x) { ok = true; break; }
            __nanosleep(20);
        }
        if (!ok) flag_error(p.status, SLIM_ERR_TIMEOUT);
        __threadfence();
        // the last CTA to leave puts the counters back to zero for the next call
        if (atomicAdd(&p.sync[1], 1u) == gridDim.x - 1) {
            p.sync[0] = 0u;
            p.sync[1] = 0u;
            __threadfence();
        }
    }
    __syncthreads();

    // ------------------------------------------------------------ phase 2
    const int r_pad = p.r_pad;
    if (p.r > 0) {
        // T = sum over k-slices of the X R^T partials, rounded to bf16, as
        // Ts[token][j]; columns r .. r_pad are zero
        for (int idx = threadIdx.x; idx < NT * 8 * (r_pad - p.r); idx += kDecodeThreads) {
            const int m = idx / (r_pad - p.r), j = p.r + idx % (r_pad - p.r);
            Ts[m * r_pad + j] = __float2bfloat16_rn(0.f);
        }
        for (int idx = threadIdx.x; idx < tilesR * frag; idx += kDecodeThreads) {
            const int jt = idx / frag, f = idx % frag;
            float sum = 0.f;
            for (int ks = 0; ks < p.KS; ++ks) sum += __ldcg(p.Tpart + ((size_t)ks * tilesR + jt) * frag + f);
            const int hq = f >> 5, ln = f & 31;
            const int h = hq >> 2, q = hq & 3;
            const int j = jt * 16 + (ln >> 2) + 8 * (q >> 1);
            const int m = 8 * h + 2 * (ln & 3) + (q & 1);
            Ts[m * r_pad + j] = __float2bfloat16_rn(sum);
        }
    }
    __syncthreads();

    for (int tile = blockIdx.x * kWarps + warp; tile < tilesW; tile += gridDim.x * kWarps) {
        float acc[NT][4];
#pragma unroll
        for (int h = 0; h < NT; ++h)
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                float sum = 0.f;
                for (int ks = 0; ks < p.KS; ++ks)
                    sum += __ldcg(p.Ppart + ((size_t)ks * tilesW + tile) * frag + (h * 4 + q) * 32 + lane);
                acc[h][q] = sum * p.s;
            }
        if (p.r > 0) {
            const __nv_bfloat16* l0 = p.L + ((size_t)tile * 16 + g) * p.r + 8 * t;
            const __nv_bfloat16* l1 = l0 + (size_t)8 * p.r;
            for (int jj = 0; jj < r_pad / 32; ++jj) {
                const int kk = 32 * jj + 8 * t;
                uint4 la = make_uint4(0, 0, 0, 0), lb = la;
                if (kk < p.r) { la = ldg_stream(l0 + 32 * jj); lb = ldg_stream(l1 + 32 * jj); }
#pragma unroll
                for (int h = 0; h < NT; ++h) {
                    const uint4 tb = *reinterpret_cast<const uint4*>(Ts + (g + 8 * h) * r_pad + kk);
                    mma_16816(acc[h], la.x, lb.x, la.y, lb.y, tb.x, tb.y);
                    mma_16816(acc[h], la.z, lb.z, la.w, lb.w, tb.z, tb.w);
                }
            }
        }
#pragma unroll
        for (int h = 0; h < NT; ++h)
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int m = 8 * h + 2 * t + (q & 1);
                const int n = tile * 16 + g + 8 * (q >> 1);
                if (m < p.b) p.Y[(size_t)m * p.d_out + n] = __float2bfloat16_rn(acc[h][q]);
            }
    }
}

// ------------------------------------------------------------------ host side
struct DecodePlan { int KS, nblk, GW, GR, r_pad, nt; size_t p_bytes, t_bytes, smem; };

static int pad_rank(int r) {
    if (r == 0) return 0;
    int rp = (r + 31) / 32 * 32;
    if (rp % 64 == 0) rp += 32;      // token rows 64 bytes apart modulo 128: conflict-free 16-byte reads
    return rp;
}

static bool make_plan(int b, int d_out, int d_in, int r, int ctas, DecodePlan* pl) {
    if (b < 1 || b > 16 || d_in % 256 != 0 || d_out % 16 != 0 || r % 16 != 0 || r > kMaxDecodeRank) return false;
    pl->nt = b <= 8 ? 1 : 2;
    pl->nblk = d_in / 256;
    pl->KS = ceil_div(pl->nblk, kWarps);
    int G = ctas / pl->KS;
    if (G < (r > 0 ? 2 : 1)) return false;
    const int tilesW = d_out / 16, tilesR = r / 16;
    if (r > 0) {
        const double bytesR = 2.0 * r * d_in, bytesW = 0.375 * (double)d_out * d_in;
        int GR = (int)(G * bytesR / (bytesR + bytesW) + 0.5);
        if (GR < 1) GR = 1;
        if (GR > G - 1) GR = G - 1;
        if (GR > tilesR) GR = tilesR;
        int GW = G - GR;
        if (GW > tilesW) GW = tilesW;
        pl->GR = GR; pl->GW = GW;
    } else {
        pl->GR = 0; pl->GW = G < tilesW ? G : tilesW;
    }
    pl->r_pad = pad_rank(r);
    const size_t frag = (size_t)pl->nt * 128 * sizeof(float);
    pl->p_bytes = (size_t)pl->KS * tilesW * frag;
    pl->t_bytes = (size_t)pl->KS * tilesR * frag;
    pl->smem = (size_t)pl->nt * 8 * pl->r_pad * sizeof(__nv_bfloat16);
    return true;
}

constexpr size_t kDecodeMaxDynSmem = 16 * (size_t)(kMaxDecodeRank + 64) * 2;

int decode_query_residency(int nt) {
    int n = 0;
    cudaError_t e1, e2;
    if (nt == 1) {
        e1 = cudaFuncSetAttribute(decode_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDecodeMaxDynSmem);
        e2 = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_kernel<1>, kDecodeThreads, kDecodeMaxDynSmem);
    } else {
        e1 = cudaFuncSetAttribute(decode_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDecodeMaxDynSmem);
        e2 = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_kernel<2>, kDecodeThreads, kDecodeMaxDynSmem);
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
    // split-K partial tiles; depends on the shape only, not on the device
    if (b < 1 || b > 16 || d_in % 256 != 0 || d_out % 16 != 0 || r % 16 != 0 || r > kMaxDecodeRank) return 0;
    const size_t frag = (size_t)(b <= 8 ? 1 : 2) * 128 * sizeof(float);
    const size_t KS = (size_t)ceil_div(d_in / 256, kWarps);
    return KS * (size_t)(d_out / 16 + r / 16) * frag;
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
    if (!make_plan(b, d_out, d_in, r, decode_ctas(nt), &pl)) return SLIM_ERR_UNSUPPORTED_SHAPE;
    DecodeParams p;
    p.X = X; p.vals = vals; p.meta = meta; p.L = L; p.R = R; p.Y = Y;
    char* base = reinterpret_cast<char*>(ws);
    p.sync = reinterpret_cast<uint32_t*>(base);
    p.Ppart = reinterpret_cast<float*>(base + SLIM_WORKSPACE_SYNC_BYTES);
    p.Tpart = reinterpret_cast<float*>(base + SLIM_WORKSPACE_SYNC_BYTES + pl.p_bytes);
    p.status = status_dev;
    p.s = s; p.b = b; p.r = r; p.d_out = d_out; p.d_in = d_in;
    p.KS = pl.KS; p.nblk = pl.nblk; p.GW = pl.GW; p.GR = pl.GR; p.r_pad = pl.r_pad;
    void* args[] = {&p};
    const dim3 grid(pl.KS * (pl.GW + pl.GR)), block(kDecodeThreads);
    cudaError_t e = nt == 1
        ? cudaLaunchCooperativeKernel((const void*)decode_kernel<1>, grid, block, args, pl.smem, st)
        : cudaLaunchCooperativeKernel((const void*)decode_kernel<2>, grid, block, args, pl.smem, st);
    count_launch(1);
    return e == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

}  // namespace slim
