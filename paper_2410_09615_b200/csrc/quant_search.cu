// SLiM-Quant: the per-tensor scale search and the quantization step (Sec. 3.1, Eq. 2-7, Algorithm 1;
// number of histogram bins: App. "Settings and Hyperparameters").  The steps and the precision of every
// decision are those include/slim.h states for slim_quant: the bin of a weight in binary32, the error
// of a candidate in binary64 with the bins added in ascending order and no fused multiply-add, the
// codes in binary32.  Four launches: largest magnitude, histogram, search, codes.
#include "common.cuh"

namespace slim {

namespace {

constexpr int kQsTable = 29;          // candidates: ten coarse, nineteen fine

struct QsHeader {                     // first 256 bytes of the workspace
    unsigned int max_bits;            // bit pattern of the largest |w| (non-negative floats order like unsigned integers)
    unsigned int bad;                 // a NaN or an infinity was seen
};

__global__ void qs_absmax_kernel(const float* __restrict__ W, size_t n, QsHeader* hdr)
{
    unsigned int m = 0, bad = 0;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float a = fabsf(W[i]);
        if (!(a <= 3.0e38f)) bad = 1;
        m = max(m, __float_as_uint(a));
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) { m = max(m, __shfl_xor_sync(0xffffffffu, m, o)); bad |= __shfl_xor_sync(0xffffffffu, bad, o); }
    if ((threadIdx.x & 31) == 0) {
        if (!bad) atomicMax(&hdr->max_bits, m);
        if (bad) atomicOr(&hdr->bad, 1u);
    }
}

// Histogram of |w| / M over `bins` uniform bins, per block in shared memory, then added to the global one.
__global__ void qs_hist_kernel(const float* __restrict__ W, size_t n, const QsHeader* hdr, int bins, unsigned int* hist)
{
    extern __shared__ unsigned int sh[];
    for (int i = threadIdx.x; i < bins; i += blockDim.x) sh[i] = 0;
    __syncthreads();
    const float M = __uint_as_float(hdr->max_bits);
    if (M > 0.f && !hdr->bad) {
        const float fb = (float)bins;
        for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
            int b = (int)__fmul_rn(__fdiv_rn(fabsf(W[i]), M), fb);
            b = min(b, bins - 1);
            atomicAdd(&sh[b], 1u);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < bins; i += blockDim.x)
        if (sh[i]) atomicAdd(&hist[i], sh[i]);
}

// E(alpha) on the bin centres, by one warp: the lanes work out the terms of 32 bins at a time, every operation
// rounded on its own, and lane 0 adds them in ascending order of the bins (an empty bin adds +0, which changes
// nothing), so the sum is the one a single thread would get.  Returns the sum in lane 0.
__device__ double qs_error(const unsigned int* hist, int bins, double M, double n_total, double alpha, double* terms, int lane)
{
    double e = 0.0;
    const double width = __ddiv_rn(M, (double)bins);
    for (int i0 = 0; i0 < bins; i0 += 32) {
        const int i = i0 + lane;
        double term = 0.0;
        const unsigned int c = i < bins ? hist[i] : 0u;
        if (c) {
            const double x = __dmul_rn(__dadd_rn((double)i, 0.5), width);
            const double p = __ddiv_rn((double)c, n_total);
            double d;
            if (x <= alpha) {
                const double level = rint(__ddiv_rn(__dmul_rn(x, 8.0), alpha));
                d = __dsub_rn(__dmul_rn(__dmul_rn(alpha, 0.125), level), x);
            } else {
                d = __dsub_rn(alpha, x);
            }
            term = __dmul_rn(p, __dmul_rn(d, d));
        }
        terms[lane] = term;
        __syncwarp();
        if (lane == 0) {
#pragma unroll
            for (int k = 0; k < 32; ++k) e = __dadd_rn(e, terms[k]);
        }
        __syncwarp();
    }
    return e;
}

// One block of 32 warps: warps 0-9 take the coarse candidates, then warps 0-18 the fine ones; thread 0 takes
// the minima in the order the algorithm visits the candidates.
__global__ void __launch_bounds__(1024, 1)
qs_search_kernel(const QsHeader* hdr, const unsigned int* hist, int bins, double n_total,
                 float* scale_alpha, double* table, uint32_t* status)
{
    __shared__ double a_s[kQsTable], e_s[kQsTable];
    __shared__ double terms[32][32];
    __shared__ double a_low_s;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float Mf = __uint_as_float(hdr->max_bits);
    if (hdr->bad || !(Mf > 0.f)) {
        if (threadIdx.x == 0) {
            scale_alpha[0] = 0.f; scale_alpha[1] = 0.f;
            if (hdr->bad) flag_error(status, SLIM_ERR_INVALID_ARG);
        }
        for (int i = threadIdx.x; i < 2 * kQsTable + 1; i += blockDim.x) table[i] = 0.0;
        return;
    }
    const double M = (double)Mf, eta_low = __ddiv_rn(M, 10.0), eta_high = __ddiv_rn(eta_low, 10.0);
    if (warp < 10) {
        const double a = __ddiv_rn(__dmul_rn(M, (double)(warp + 1)), 10.0);
        const double e = qs_error(hist, bins, M, n_total, a, terms[warp], lane);
        if (lane == 0) { a_s[warp] = a; e_s[warp] = e; }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int best = 0;
        for (int k = 1; k < 10; ++k) if (e_s[k] < e_s[best]) best = k;
        a_low_s = a_s[best];
    }
    __syncthreads();
    if (warp < 19) {
        double a = __dadd_rn(__dsub_rn(a_low_s, eta_low), __dmul_rn((double)(warp + 1), eta_high));
        if (a > M) a = M;
        const double e = a > 0.0 ? qs_error(hist, bins, M, n_total, a, terms[warp], lane) : -1.0;
        if (lane == 0) { a_s[10 + warp] = a; e_s[10 + warp] = e; }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double best_a = a_s[0], best_e = e_s[0];
        for (int k = 1; k < 10; ++k) if (e_s[k] < best_e) { best_a = a_s[k]; best_e = e_s[k]; }
        for (int j = 10; j < kQsTable; ++j) {
            if (!(a_s[j] > 0.0)) { e_s[j] = __dadd_rn(best_e, 1.0); continue; }     // not a candidate; listed like this
            if (e_s[j] < best_e || (e_s[j] == best_e && a_s[j] < best_a)) { best_a = a_s[j]; best_e = e_s[j]; }
        }
        const float a32 = (float)best_a;
        scale_alpha[0] = __fmul_rn(a32, 0.125f);
        scale_alpha[1] = a32;
        table[2 * kQsTable] = best_a;
    }
    __syncthreads();
    if (threadIdx.x < kQsTable) { table[2 * threadIdx.x] = a_s[threadIdx.x]; table[2 * threadIdx.x + 1] = e_s[threadIdx.x]; }
}

__global__ void qs_codes_kernel(const float* __restrict__ W, size_t n, const float* __restrict__ scale_alpha, int8_t* __restrict__ codes)
{
    const float a32 = scale_alpha[1];
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        int q = 0;
        if (a32 > 0.f) q = max(-8, min(7, __float2int_rn(__fmul_rn(__fdiv_rn(W[i], a32), 8.0f))));
        codes[i] = (int8_t)q;
    }
}

}  // namespace

int quant_bins(int d_out, int d_in) {
    long long b = (long long)d_out * (long long)d_in / 1000;
    if (b > 20000) b = 20000;
    if (b < 512) b = 512;
    return (int)b;
}

size_t quant_workspace_bytes(int d_out, int d_in) {
    return 256 + (size_t)quant_bins(d_out, d_in) * 4 + 256 + (2 * kQsTable + 1) * sizeof(double);
}

slim_status_t launch_quant(const float* W, int d_out, int d_in, int8_t* codes, float* scale_alpha, void* ws,
                           uint32_t* status_dev, cudaStream_t st)
{
    slim_status_t err;
    const DeviceInfo* di = device_info(&err);
    if (!di) return err;
    const size_t n = (size_t)d_out * (size_t)d_in;
    const int bins = quant_bins(d_out, d_in);
    char* base = static_cast<char*>(ws);
    QsHeader* hdr = reinterpret_cast<QsHeader*>(base);
    unsigned int* hist = reinterpret_cast<unsigned int*>(base + 256);
    double* table = reinterpret_cast<double*>(base + 256 + ((size_t)bins * 4 + 255) / 256 * 256);
    if (cudaMemsetAsync(ws, 0, 256 + (size_t)bins * 4, st) != cudaSuccess) return SLIM_ERR_CUDA;
    const unsigned grid = (unsigned)(di->sm_count * 4);
    qs_absmax_kernel<<<grid, 512, 0, st>>>(W, n, hdr);
    const size_t hist_smem = (size_t)bins * 4;
    if (hist_smem > 48 * 1024 &&
        cudaFuncSetAttribute(qs_hist_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)hist_smem) != cudaSuccess)
        return SLIM_ERR_CUDA;
    qs_hist_kernel<<<(unsigned)(di->sm_count * 2), 1024, hist_smem, st>>>(W, n, hdr, bins, hist);
    qs_search_kernel<<<1, 1024, 0, st>>>(hdr, hist, bins, (double)n, scale_alpha, table, status_dev);
    qs_codes_kernel<<<grid, 512, 0, st>>>(W, n, scale_alpha, codes);
    count_launch(4);
    return cudaGetLastError() == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

}  // namespace slim
