// C-ABI entry points of libslim: argument checks, dispatch by batch size,
// per-device attribute cache.  All arithmetic lives in the kernel files.
#include <atomic>
#include <cmath>
#include <mutex>
#include "common.cuh"

namespace slim {

static DeviceInfo g_info[64];
static std::atomic<bool> g_info_ready[64];
static std::mutex g_info_mutex;
static thread_local int t_launches = 0;
static thread_local int t_token_tile = 0;

void count_launch(int n) { t_launches += n; }
void reset_launch_count() { t_launches = 0; t_token_tile = 0; }
void note_token_tile(int n) { t_token_tile = n; }

// The record of a device is filled once under the mutex and published with a release store;
// readers take it with an acquire load, so they never see a half-written record.
const DeviceInfo* device_info(slim_status_t* err) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { *err = SLIM_ERR_CUDA; return nullptr; }
    DeviceInfo& di = g_info[dev];
    if (!g_info_ready[dev].load(std::memory_order_acquire)) {
        std::lock_guard<std::mutex> lock(g_info_mutex);
        if (!g_info_ready[dev].load(std::memory_order_relaxed)) {
            cudaDeviceProp prop;
            if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { *err = SLIM_ERR_CUDA; return nullptr; }
            di.cc_major = prop.major;
            di.sm_count = prop.multiProcessorCount;
            if (prop.major == 10) {
                di.decode_ctas_per_sm[0] = decode_query_residency(1);
                di.decode_ctas_per_sm[1] = decode_query_residency(2);
                di.decode_tiled_ok = decode_tiled_query_residency();
            }
            g_info_ready[dev].store(true, std::memory_order_release);
        }
    }
    if (di.cc_major != 10) { *err = SLIM_ERR_ARCH; return nullptr; }
    return &di;
}

void* tensor_map_encoder() {
    static std::atomic<void*> cached{nullptr};
    void* fn = cached.load(std::memory_order_acquire);
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess && ptr) {
            cached.store(ptr, std::memory_order_release);      // every thread finds the same address
            fn = ptr;
        }
    }
    return fn;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static slim_status_t check_weight_shape(int d_out, int d_in) {
    if (d_out < 1 || d_in < 1) return SLIM_ERR_INVALID_ARG;
    if (d_in % 64 != 0 || d_out % 16 != 0) return SLIM_ERR_UNSUPPORTED_SHAPE;
    return SLIM_OK;
}

static slim_kernel_t select_kernel(int b, int d_out, int d_in, int r) {
    if (b <= 16 && decode_supports(b, d_out, d_in, r)) return SLIM_KERNEL_DECODE;
    if (b > 16 && prefill_supports(b, d_out, d_in, r)) return SLIM_KERNEL_PREFILL;
    return SLIM_KERNEL_SIMPLE;
}

static size_t workspace_bytes(int b, int d_out, int d_in, int r) {
    size_t need = simple_workspace_bytes(b, d_out, d_in, r);
    const size_t d = decode_workspace_bytes(b, d_out, d_in, r);
    if (d > need) need = d;
    const size_t pf = prefill_workspace_bytes(b, d_out, d_in, r);
    if (pf > need) need = pf;
    const size_t dt = b <= 16 ? decode_tiled_workspace_bytes(b, d_out, d_in, r) : 0;
    if (dt > need) need = dt;
    need = (need + 255) / 256 * 256;
    return SLIM_WORKSPACE_SYNC_BYTES + need;
}

}  // namespace slim

using namespace slim;

extern "C" {

slim_status_t slim_pack(const int8_t* codes, const uint8_t* mask, int d_out, int d_in,
                        uint8_t* vals, uint8_t* meta, uint32_t* status_dev, void* cuda_stream)
{
    reset_launch_count();
    if (!codes || !mask || !vals || !meta) return SLIM_ERR_INVALID_ARG;
    slim_status_t st = check_weight_shape(d_out, d_in);
    if (st != SLIM_OK) return st;
    if (!aligned16(codes) || !aligned16(mask) || !aligned16(vals) || !aligned16(meta)) return SLIM_ERR_INVALID_ARG;
    if (status_dev && (reinterpret_cast<uintptr_t>(status_dev) & 3u)) return SLIM_ERR_INVALID_ARG;
    return launch_pack(codes, mask, d_out, d_in, vals, meta, status_dev, (cudaStream_t)cuda_stream);
}

slim_status_t slim_unpack(const uint8_t* vals, const uint8_t* meta, int d_out, int d_in,
                          int8_t* codes, uint8_t* mask, void* cuda_stream)
{
    reset_launch_count();
    if (!vals || !meta || !codes) return SLIM_ERR_INVALID_ARG;
    slim_status_t st = check_weight_shape(d_out, d_in);
    if (st != SLIM_OK) return st;
    if (!aligned16(codes) || !aligned16(vals) || !aligned16(meta) || (mask && !aligned16(mask))) return SLIM_ERR_INVALID_ARG;
    return launch_unpack(vals, meta, d_out, d_in, codes, mask, (cudaStream_t)cuda_stream);
}

size_t slim_workspace_bytes(int b, int d_out, int d_in, int r)
{
    if (b < 1 || r < 0 || r % 16 != 0 || check_weight_shape(d_out, d_in) != SLIM_OK) return 0;
    return workspace_bytes(b, d_out, d_in, r);
}

slim_status_t slim_workspace_reset(void* workspace, size_t workspace_bytes_, void* cuda_stream)
{
    if (!workspace || workspace_bytes_ < SLIM_WORKSPACE_SYNC_BYTES) return SLIM_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // hand-over slots start "empty" (all-ones), the call counter at zero
    if (cudaMemsetAsync(workspace, 0xFF, workspace_bytes_, st) != cudaSuccess) return SLIM_ERR_CUDA;
    return cudaMemsetAsync(workspace, 0, SLIM_WORKSPACE_SYNC_BYTES, st) == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

int slim_decode_layout_hint(int b, int d_out, int d_in, int r)
{
    if (b < 1 || b > (d_out >= d_in ? 4 : 2) || r < 0 || r % 16 != 0 || check_weight_shape(d_out, d_in) != SLIM_OK) return 0;
    if ((size_t)d_out * (size_t)d_in * 3 / 8 < ((size_t)64 << 20)) return 0;
    slim_status_t err;
    const DeviceInfo* di = device_info(&err);
    if (!di || !di->decode_tiled_ok || !decode_tiled_supports(b, d_out, d_in, r)) return 0;
    return SLIM_LAYOUT_DECODE_TILED;
}

slim_kernel_t slim_select_kernel(int b, int d_out, int d_in, int r)
{
    if (b < 1 || r < 0 || r % 16 != 0 || check_weight_shape(d_out, d_in) != SLIM_OK) return SLIM_KERNEL_AUTO;
    return select_kernel(b, d_out, d_in, r);
}

slim_status_t slim_linear_fwd_ex(const void* X, int b, const uint8_t* vals, const uint8_t* meta,
                                 float s, const void* L, const void* R, int r, int d_out, int d_in,
                                 void* Y, void* workspace, size_t workspace_bytes_,
                                 uint32_t* status_dev, void* cuda_stream, slim_kernel_t kernel)
{
    reset_launch_count();
    if (!X || !vals || !meta || !Y || b < 1 || r < 0 || !std::isfinite(s)) return SLIM_ERR_INVALID_ARG;
    if ((r > 0) != (L != nullptr) || (r > 0) != (R != nullptr)) return SLIM_ERR_INVALID_ARG;
    slim_status_t st = check_weight_shape(d_out, d_in);
    if (st != SLIM_OK) return st;
    if (r % 16 != 0) return SLIM_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(X) || !aligned16(vals) || !aligned16(meta) || !aligned16(Y) || !aligned16(L) || !aligned16(R) ||
        !aligned16(workspace))
        return SLIM_ERR_INVALID_ARG;
    if (status_dev && (reinterpret_cast<uintptr_t>(status_dev) & 3u)) return SLIM_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes_ < workspace_bytes(b, d_out, d_in, r)) return SLIM_ERR_WORKSPACE;
    slim_status_t derr;
    if (!device_info(&derr)) return derr;
    if (kernel == SLIM_KERNEL_AUTO) kernel = select_kernel(b, d_out, d_in, r);
    const __nv_bfloat16* Xb = static_cast<const __nv_bfloat16*>(X);
    const __nv_bfloat16* Lb = static_cast<const __nv_bfloat16*>(L);
    const __nv_bfloat16* Rb = static_cast<const __nv_bfloat16*>(R);
    __nv_bfloat16* Yb = static_cast<__nv_bfloat16*>(Y);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    switch (kernel) {
    case SLIM_KERNEL_SIMPLE:
        return launch_simple(Xb, b, vals, meta, s, Lb, Rb, r, d_out, d_in, Yb, workspace, stream);
    case SLIM_KERNEL_DECODE:
        if (b > 16 || !decode_supports(b, d_out, d_in, r)) return SLIM_ERR_UNSUPPORTED_SHAPE;
        return launch_decode(Xb, b, vals, meta, s, Lb, Rb, r, d_out, d_in, Yb, workspace, status_dev, stream);
    case SLIM_KERNEL_PREFILL:
        if (!prefill_supports(b, d_out, d_in, r)) return SLIM_ERR_UNSUPPORTED_SHAPE;
        return launch_prefill(Xb, b, vals, meta, s, Lb, Rb, r, d_out, d_in, Yb, workspace, status_dev, stream);
    case SLIM_KERNEL_PREFILL_PAIR:
        if (!prefill_supports(b, d_out, d_in, r)) return SLIM_ERR_UNSUPPORTED_SHAPE;
        return launch_prefill(Xb, b, vals, meta, s, Lb, Rb, r, d_out, d_in, Yb, workspace, status_dev, stream, true);
    default:
        return SLIM_ERR_UNSUPPORTED_SHAPE;
    }
}

slim_status_t slim_linear_fwd(const void* X, int b, const uint8_t* vals, const uint8_t* meta,
                              float s, const void* L, const void* R, int r, int d_out, int d_in,
                              void* Y, void* workspace, size_t workspace_bytes_,
                              uint32_t* status_dev, void* cuda_stream)
{
    return slim_linear_fwd_ex(X, b, vals, meta, s, L, R, r, d_out, d_in, Y, workspace, workspace_bytes_,
                              status_dev, cuda_stream, SLIM_KERNEL_AUTO);
}

size_t slim_quant_workspace_bytes(int d_out, int d_in)
{
    return d_out < 1 || d_in < 1 ? 0 : quant_workspace_bytes(d_out, d_in);
}

slim_status_t slim_quant(const float* W, int d_out, int d_in, int8_t* codes, float* scale_alpha, void* workspace,
                         size_t workspace_bytes_, uint32_t* status_dev, void* cuda_stream)
{
    reset_launch_count();
    if (!W || !codes || !scale_alpha || d_out < 1 || d_in < 1) return SLIM_ERR_INVALID_ARG;
    if (!aligned16(W) || !aligned16(codes) || !aligned16(scale_alpha) || !aligned16(workspace)) return SLIM_ERR_INVALID_ARG;
    if (status_dev && (reinterpret_cast<uintptr_t>(status_dev) & 3u)) return SLIM_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes_ < quant_workspace_bytes(d_out, d_in)) return SLIM_ERR_WORKSPACE;
    return launch_quant(W, d_out, d_in, codes, scale_alpha, workspace, status_dev, (cudaStream_t)cuda_stream);
}

slim_status_t slim_mask_top2(const int8_t* codes, const float* xbar, int d_out, int d_in, uint8_t* mask, uint32_t* status_dev,
                             void* cuda_stream)
{
    reset_launch_count();
    if (!codes || !mask || d_out < 1 || d_in < 4) return SLIM_ERR_INVALID_ARG;
    if (d_in % 4 != 0) return SLIM_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(codes) || !aligned16(mask) || !aligned16(xbar)) return SLIM_ERR_INVALID_ARG;
    if (status_dev && (reinterpret_cast<uintptr_t>(status_dev) & 3u)) return SLIM_ERR_INVALID_ARG;
    return launch_mask_top2(codes, xbar, d_out, d_in, mask, status_dev, (cudaStream_t)cuda_stream);
}

size_t slim_adapter_code_bytes(int rows, int cols)
{
    return rows < 1 || cols < 2 || cols % 2 != 0 ? 0 : (size_t)rows * (size_t)(cols / 2);
}

size_t slim_adapter_scale_bytes(int rows, int cols)
{
    return rows < 1 || cols < 2 || cols % 2 != 0 ? 0 : (size_t)rows * (size_t)((cols + 127) / 128) * 2;
}

slim_status_t slim_pack_adapter(const void* A, int rows, int cols, uint8_t* codes, void* scales, void* cuda_stream)
{
    reset_launch_count();
    if (!A || !codes || !scales || slim_adapter_code_bytes(rows, cols) == 0) return SLIM_ERR_INVALID_ARG;
    if (!aligned16(A) || !aligned16(codes) || !aligned16(scales)) return SLIM_ERR_INVALID_ARG;
    return launch_pack_adapter(static_cast<const __nv_bfloat16*>(A), rows, cols, codes, static_cast<__nv_bfloat16*>(scales),
                               (cudaStream_t)cuda_stream);
}

slim_status_t slim_unpack_adapter(const uint8_t* codes, const void* scales, int rows, int cols, void* A_out, void* cuda_stream)
{
    reset_launch_count();
    if (!A_out || !codes || !scales || slim_adapter_code_bytes(rows, cols) == 0) return SLIM_ERR_INVALID_ARG;
    if (!aligned16(A_out) || !aligned16(codes) || !aligned16(scales)) return SLIM_ERR_INVALID_ARG;
    return launch_unpack_adapter(codes, static_cast<const __nv_bfloat16*>(scales), rows, cols, static_cast<__nv_bfloat16*>(A_out),
                                 (cudaStream_t)cuda_stream);
}

static size_t align256(size_t n) { return (n + 255) / 256 * 256; }

size_t slim_workspace_bytes_q(int b, int d_out, int d_in, int r)
{
    const size_t base = slim_workspace_bytes(b, d_out, d_in, r);
    if (base == 0 || r < 16) return 0;
    return align256(base) + align256((size_t)d_out * r * 2) + align256((size_t)r * d_in * 2);
}

slim_status_t slim_linear_fwd_q(const void* X, int b, const uint8_t* vals, const uint8_t* meta, float s,
                                const uint8_t* Lq, const void* Ls, const uint8_t* Rq, const void* Rs, int r,
                                int d_out, int d_in, void* Y, void* workspace, size_t workspace_bytes_,
                                uint32_t* status_dev, void* cuda_stream)
{
    reset_launch_count();
    if (!Lq || !Ls || !Rq || !Rs || r < 16 || r % 16 != 0) return SLIM_ERR_INVALID_ARG;
    if (!aligned16(Lq) || !aligned16(Ls) || !aligned16(Rq) || !aligned16(Rs) || !aligned16(workspace)) return SLIM_ERR_INVALID_ARG;
    const size_t need = slim_workspace_bytes_q(b, d_out, d_in, r);
    if (need == 0) return SLIM_ERR_UNSUPPORTED_SHAPE;
    if (!workspace || workspace_bytes_ < need) return SLIM_ERR_WORKSPACE;
    const size_t base = align256(slim_workspace_bytes(b, d_out, d_in, r));
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // small batches: the decode kernel reads the codes and scales as they are
    if (b <= 16 && decode_supports_q(b, d_out, d_in, r)) {
        if (!X || !vals || !meta || !Y || !std::isfinite(s)) return SLIM_ERR_INVALID_ARG;
        if (!aligned16(X) || !aligned16(vals) || !aligned16(meta) || !aligned16(Y)) return SLIM_ERR_INVALID_ARG;
        if (status_dev && (reinterpret_cast<uintptr_t>(status_dev) & 3u)) return SLIM_ERR_INVALID_ARG;
        slim_status_t derr;
        if (!device_info(&derr)) return derr;
        return launch_decode_q(static_cast<const __nv_bfloat16*>(X), b, vals, meta, s, Lq, static_cast<const __nv_bfloat16*>(Ls), Rq,
                               static_cast<const __nv_bfloat16*>(Rs), r, d_out, d_in, static_cast<__nv_bfloat16*>(Y), workspace,
                               status_dev, st);
    }
    char* w = static_cast<char*>(workspace);
    __nv_bfloat16* Ld = reinterpret_cast<__nv_bfloat16*>(w + base);
    __nv_bfloat16* Rd = reinterpret_cast<__nv_bfloat16*>(w + base + align256((size_t)d_out * r * 2));
    slim_status_t rc = launch_unpack_adapter(Lq, static_cast<const __nv_bfloat16*>(Ls), d_out, r, Ld, st);
    if (rc == SLIM_OK) rc = launch_unpack_adapter(Rq, static_cast<const __nv_bfloat16*>(Rs), r, d_in, Rd, st);
    if (rc != SLIM_OK) return rc;
    const int dequant_launches = slim_last_launch_count();
    rc = slim_linear_fwd_ex(X, b, vals, meta, s, Ld, Rd, r, d_out, d_in, Y, workspace, base, status_dev, cuda_stream,
                            SLIM_KERNEL_AUTO);
    count_launch(dequant_launches);
    return rc;
}

size_t slim_tiled_bytes(int d_out, int d_in, int layout_id)
{
    if (layout_id != SLIM_LAYOUT_DECODE_TILED || d_out < 16 || d_in < 256 || d_out % 16 != 0 || d_in % 256 != 0) return 0;
    return (size_t)((d_out + 63) / 64 * 64) * (size_t)d_in / 8 * 3;       // whole groups of four 16-row tiles
}

slim_status_t slim_repack_tiled(const uint8_t* vals, const uint8_t* meta, int d_out, int d_in, int layout_id,
                                void* tiled_out, void* cuda_stream)
{
    reset_launch_count();
    if (!vals || !meta || !tiled_out || d_out < 1 || d_in < 1) return SLIM_ERR_INVALID_ARG;
    if (slim_tiled_bytes(d_out, d_in, layout_id) == 0) return SLIM_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(vals) || !aligned16(meta) || !aligned16(tiled_out)) return SLIM_ERR_INVALID_ARG;
    return launch_repack_tiled(vals, meta, d_out, d_in, static_cast<uint8_t*>(tiled_out), (cudaStream_t)cuda_stream);
}

slim_status_t slim_linear_fwd_tiled(const void* X, int b, const void* tiled, int layout_id, float s, const void* L,
                                    const void* R, int r, int d_out, int d_in, void* Y, void* workspace,
                                    size_t workspace_bytes_, uint32_t* status_dev, void* cuda_stream)
{
    reset_launch_count();
    if (!X || !tiled || !Y || b < 1 || r < 0 || d_out < 1 || d_in < 1 || !std::isfinite(s)) return SLIM_ERR_INVALID_ARG;
    if ((r > 0) != (L != nullptr) || (r > 0) != (R != nullptr)) return SLIM_ERR_INVALID_ARG;
    if (slim_tiled_bytes(d_out, d_in, layout_id) == 0 || r % 16 != 0 || b > 16) return SLIM_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(X) || !aligned16(tiled) || !aligned16(Y) || !aligned16(L) || !aligned16(R) || !aligned16(workspace))
        return SLIM_ERR_INVALID_ARG;
    if (status_dev && (reinterpret_cast<uintptr_t>(status_dev) & 3u)) return SLIM_ERR_INVALID_ARG;
    slim_status_t derr;
    if (!device_info(&derr)) return derr;
    if (!decode_tiled_supports(b, d_out, d_in, r)) return SLIM_ERR_UNSUPPORTED_SHAPE;
    if (!workspace || workspace_bytes_ < workspace_bytes(b, d_out, d_in, r)) return SLIM_ERR_WORKSPACE;
    return launch_decode_tiled(static_cast<const __nv_bfloat16*>(X), b, static_cast<const uint8_t*>(tiled), s,
                               static_cast<const __nv_bfloat16*>(L), static_cast<const __nv_bfloat16*>(R), r, d_out, d_in,
                               static_cast<__nv_bfloat16*>(Y), workspace, status_dev, (cudaStream_t)cuda_stream);
}

slim_status_t slim_linear_fwd_tiled_host(const void* X_host, int b, const void* tiled, int layout_id, float s,
                                         const void* L, const void* R, int r, int d_out, int d_in, void* Y_host,
                                         void* x_dev, void* y_dev, void* workspace, size_t workspace_bytes_,
                                         uint32_t* status_dev, void* cuda_stream)
{
    if (!X_host || !Y_host || !x_dev || !y_dev || b < 1 || d_in < 1 || d_out < 1) return SLIM_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(x_dev, X_host, (size_t)b * d_in * 2, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return SLIM_ERR_CUDA;
    slim_status_t st = slim_linear_fwd_tiled(x_dev, b, tiled, layout_id, s, L, R, r, d_out, d_in, y_dev, workspace,
                                             workspace_bytes_, status_dev, cuda_stream);
    if (st != SLIM_OK) return st;
    if (cudaMemcpyAsync(Y_host, y_dev, (size_t)b * d_out * 2, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return SLIM_ERR_CUDA;
    return cudaStreamSynchronize(stream) == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

slim_status_t slim_linear_fwd_host(const void* X_host, int b, const uint8_t* vals,
                                   const uint8_t* meta, float s, const void* L, const void* R,
                                   int r, int d_out, int d_in, void* Y_host, void* x_dev,
                                   void* y_dev, void* workspace, size_t workspace_bytes_,
                                   uint32_t* status_dev, void* cuda_stream)
{
    if (!X_host || !Y_host || !x_dev || !y_dev || b < 1 || d_in < 1 || d_out < 1) return SLIM_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(x_dev, X_host, (size_t)b * d_in * 2, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return SLIM_ERR_CUDA;
    slim_status_t st = slim_linear_fwd(x_dev, b, vals, meta, s, L, R, r, d_out, d_in, y_dev, workspace,
                                       workspace_bytes_, status_dev, cuda_stream);
    if (st != SLIM_OK) return st;
    if (cudaMemcpyAsync(Y_host, y_dev, (size_t)b * d_out * 2, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return SLIM_ERR_CUDA;
    return cudaStreamSynchronize(stream) == cudaSuccess ? SLIM_OK : SLIM_ERR_CUDA;
}

int slim_last_launch_count(void) { return t_launches; }

int slim_last_token_tile(void) { return t_token_tile; }

const char* slim_strerror(slim_status_t status)
{
    switch (status) {
    case SLIM_OK: return "ok";
    case SLIM_ERR_INVALID_ARG: return "invalid argument (null or misaligned pointer, bad size)";
    case SLIM_ERR_UNSUPPORTED_SHAPE: return "unsupported shape (d_in % 64, d_out % 16, r % 16 must be 0)";
    case SLIM_ERR_BAD_MASK: return "a 2:4 group keeps more than two values";
    case SLIM_ERR_CODE_RANGE: return "a kept code lies outside [-8, 7]";
    case SLIM_ERR_WORKSPACE: return "workspace missing or too small";
    case SLIM_ERR_CUDA: return "CUDA runtime error";
    case SLIM_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case SLIM_ERR_ARCH: return "device is not compute capability 10.x";
    }
    return "unknown status";
}

const char* slim_version(void) { return "libslim 0.2 (sm_100a)"; }

}  // extern "C"
