/*
 * libslim — the SLiM compressed linear layer on NVIDIA B200 (sm_100a).
 *
 *     Y = X (s Q)^T + (X R^T) L^T
 *
 * Q holds symmetric-uniform 4-bit integer codes with one scale s per tensor
 * (paper Sec. 3.1, Eq. 2 / Eq. 5), pruned to the 2:4 pattern: at most two kept
 * values in every aligned group of four along d_in (Sec. 1, Sec. 3.2).  L and R
 * are the rank-r adapters that correct the compression error, W ~ W^C + L R
 * (Sec. 3.2); the layer output is Y = X W (Sec. 2, Eq. 1) and the adapter product
 * is evaluated factored, at O(2 b r d^2) cost (App. "Rank Analysis").
 *
 * Orientation (nn.Linear, the transpose of the paper's W in R^{d_in x d_out}):
 *   X [b, d_in]  bf16 row-major          activations, b tokens
 *   Q [d_out, d_in] int4 codes           row n = output feature n
 *   L [d_out, r] bf16 row-major          (the paper's right adapter, transposed)
 *   R [r, d_in]  bf16 row-major          (the paper's left adapter, transposed)
 *   Y [b, d_out] bf16 row-major
 *
 * Packed weight (the paper leaves storage to a third-party kernel; this is the
 * library's own format):
 *   vals [d_out, d_in/4] u8   one byte per group of four columns: low nibble =
 *                             code at the lower stored position, high nibble =
 *                             code at the upper one (two's complement)
 *   meta [d_out, d_in/8] u8   one nibble per group: bits 0-1 lower position,
 *                             bits 2-3 upper position (lower < upper); even
 *                             groups in the low nibble of a byte
 *   A group with fewer than two kept positions is completed with the lowest
 *   positions not kept, stored with value 0.
 *
 * General rules for every call:
 *   - Every data pointer is a DEVICE pointer owned by the caller and must be
 *     16-byte aligned; the library allocates no device memory and keeps no
 *     state besides a per-device attribute cache.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL =
 *     the default stream) and the call returns without synchronising.
 *   - The return value reports errors the host can see (bad arguments,
 *     unsupported shape or device, a failed launch).  Errors found on the
 *     device (a 2:4 group with more than two kept values, a code outside
 *     [-8, 7], a bounded wait that expired) are OR-ed as bits
 *     (1u << slim_status_t) into *status_dev, a device uint32 the caller
 *     zeroes and reads back; status_dev may be NULL.  Nothing traps.
 */
#ifndef SLIM_H
#define SLIM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SLIM_OK = 0,
    SLIM_ERR_INVALID_ARG = 1,        /* null / misaligned pointer, b < 1, negative size, scale not finite */
    SLIM_ERR_UNSUPPORTED_SHAPE = 2,  /* d_in % 64, d_out % 16 or r % 16 not zero */
    SLIM_ERR_BAD_MASK = 3,           /* device: more than two kept values in a group */
    SLIM_ERR_CODE_RANGE = 4,         /* device: kept code outside [-8, 7] */
    SLIM_ERR_WORKSPACE = 5,          /* workspace NULL or smaller than slim_workspace_bytes */
    SLIM_ERR_CUDA = 6,               /* a CUDA runtime call or launch failed */
    SLIM_ERR_TIMEOUT = 7,            /* device: a bounded wait expired */
    SLIM_ERR_ARCH = 8                /* current device is not compute capability 10.x */
} slim_status_t;

/* Kernel families the dispatcher chooses from (slim_linear_fwd_ex). */
typedef enum {
    SLIM_KERNEL_AUTO = 0,    /* by batch size: decode for b <= 16, prefill above */
    SLIM_KERNEL_SIMPLE = 1,  /* CUDA-core kernel, any legal shape; correctness anchor */
    SLIM_KERNEL_DECODE = 2,  /* streaming sparse tensor-core kernel for small batches */
    SLIM_KERNEL_PREFILL = 3, /* tcgen05 sparse tensor-core kernel for many tokens */
    SLIM_KERNEL_PREFILL_PAIR = 4 /* the same with two CTAs per 256-row tile (cta_group::2); never chosen
                                    by the dispatcher; needs an even number of 128-row tiles */
} slim_kernel_t;

/*
 * Pack int4 codes and a 2:4 mask into `vals` and `meta` (format above; 2:4
 * pattern: Sec. 1; 4-bit symmetric codes: Sec. 3.1 Eq. 2).  Integer-only and
 * bit-exact.
 *   codes [d_out, d_in] int8, values in [-8, 7] at kept positions (others ignored)
 *   mask  [d_out, d_in] u8, non-zero = kept
 *   vals  [d_out, d_in/4] u8 (out),  meta [d_out, d_in/8] u8 (out)
 * d_in must be a multiple of 64.  Groups that violate the 2:4 pattern or hold an
 * out-of-range code are written as zeros (value 0x00, index nibble 0x4) and
 * flagged in *status_dev.
 */
slim_status_t slim_pack(const int8_t* codes, const uint8_t* mask, int d_out, int d_in,
                        uint8_t* vals, uint8_t* meta, uint32_t* status_dev, void* cuda_stream);

/*
 * Inverse of slim_pack (reads the packed format described at the top of this file; 2:4
 * pattern: Sec. 1; 4-bit codes: Sec. 3.1 Eq. 2): dense int8 codes (0 where nothing is
 * stored) and a mask holding 1 at the two stored positions of every group.  `mask` may be NULL.
 */
slim_status_t slim_unpack(const uint8_t* vals, const uint8_t* meta, int d_out, int d_in,
                          int8_t* codes, uint8_t* mask, void* cuda_stream);

/*
 * Bytes of device scratch slim_linear_fwd needs for this problem (split-K
 * partial sums, the adapter intermediate T = X R^T, and a call counter).
 * Returns 0 for illegal arguments.  A workspace must be initialised once with
 * slim_workspace_reset before its first use (counter zero, every hand-over slot
 * marked empty); each call, whichever kernel it runs, leaves it ready for the next
 * one, of any shape the workspace is large enough for, unless it reported
 * SLIM_ERR_TIMEOUT, after which it must be reset again.  Calls that share a
 * workspace must not overlap on the GPU.
 */
#define SLIM_WORKSPACE_SYNC_BYTES 256
size_t slim_workspace_bytes(int b, int d_out, int d_in, int r);

/* Initialise a whole workspace (asynchronous, on the stream). */
slim_status_t slim_workspace_reset(void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The layer forward (Sec. 2 Eq. 1 with W ~ W^C + L R, Sec. 3.2; factored
 * adapter product, App. "Rank Analysis"):
 *     Y[m][n] = s * sum_k X[m][k] Q[n][k]  +  sum_j (sum_k X[m][k] R[j][k]) L[n][j]
 * Products are bf16 x bf16 accumulated in fp32; the intermediate T = X R^T may
 * be rounded once to bf16; Y is rounded to bf16 (nearest even).
 *   X [b, d_in] bf16, vals/meta as produced by slim_pack, s fp32 scale,
 *   L [d_out, r] bf16, R [r, d_in] bf16 (both NULL iff r == 0), Y [b, d_out] bf16 (out).
 * Shape rules: b >= 1, d_in % 64 == 0, d_out % 16 == 0, r % 16 == 0; s must be finite
 * (NaN or infinity: SLIM_ERR_INVALID_ARG).
 * The kernel is chosen from b and the shape: for b <= 16 the streaming decode kernel, which
 * needs d_in % 256 == 0; above, the tcgen05 prefill kernel, which needs d_in % 128 == 0 and
 * d_out % 128 == 0.  Every other legal shape runs on a plain CUDA-core kernel (one warp per
 * output element) that is orders of magnitude slower: it exists for correctness, not speed.
 * For b <= 16 the fast path is slim_linear_fwd_tiled on the decode-tiled copy of the weight.
 */
slim_status_t slim_linear_fwd(const void* X, int b, const uint8_t* vals, const uint8_t* meta,
                              float s, const void* L, const void* R, int r, int d_out, int d_in,
                              void* Y, void* workspace, size_t workspace_bytes,
                              uint32_t* status_dev, void* cuda_stream);

/* Same operation with the kernel family forced (tests, benchmarks). */
slim_status_t slim_linear_fwd_ex(const void* X, int b, const uint8_t* vals, const uint8_t* meta,
                                 float s, const void* L, const void* R, int r, int d_out, int d_in,
                                 void* Y, void* workspace, size_t workspace_bytes,
                                 uint32_t* status_dev, void* cuda_stream, slim_kernel_t kernel);

/*
 * Decode-tiled copy of a packed weight, and the small-batch forward that reads it.
 *
 * At batch sizes 1-16 the layer is bound by the bytes of the weight it streams (Sec. 4
 * "Speedup": small decode batches; Fig. 3: quantization contributes most of the speed-up),
 * and the kernel then has about one instruction slot per three weight bytes.  The packed
 * format above keeps a row's bytes together, which costs the streaming kernel a byte-pick per
 * register and four-fold redundant shared-memory reads; the tiled copy holds the same nibbles
 * and position indices (0.375 byte per weight, nothing is computed) in the order the sparse
 * tensor-core instruction consumes them.  Like the packed format it is this library's own
 * layout (the paper leaves storage to a third-party kernel).  Layout SLIM_LAYOUT_DECODE_TILED,
 * for d_out % 16 == 0 and d_in % 256 == 0:
 *   the matrix is cut into tiles of 16 rows and blocks of 256 columns; (tile, block) occupies
 *   1536 bytes.  Tiles are stored in groups of four: group g = tile / 4 starts at
 *   4 g * (d_in / 256) * 1536; inside a group the blocks follow each other and inside a block the
 *   group's four tiles, so (tile, block) sits at (4 g * (d_in / 256) + block * 4 + (tile - 4 g)) * 1536
 *   and the 64 rows x 256 columns a group holds of one block are 6144 contiguous bytes (one copy
 *   request of the streaming kernel: a request costs the same issue time whatever its size).  When
 *   d_out / 16 is not a multiple of four, the last group is completed with padding pieces (value words
 *   0, every index nibble 4: stored zeros), so the buffer holds ceil(d_out / 64) * 64 rows.
 *   Inside a (tile, block) piece a "step"
 *   j = 0..7 is 32 columns (8 groups of four) and a "lane" is (g, t) = (lane / 4, lane % 4), lane = 0..31.
 *   Value words, bytes [0, 1024): the 32-bit word of (j, lane) sits at
 *   (j / 4) * 512 + lane * 16 + (j % 4) * 4 and holds four value bytes B_i, i = 0..3, of row
 *   16 tile + g + 8 (i % 2), group 8 j + 4 (i / 2) + t of the block: low nibble of B_i at bits
 *   [4 i, 4 i + 3], high nibble at bits [16 + 4 i, 16 + 4 i + 3].
 *   Index words, bytes [1024, 1536): the word of (lane, jj), jj = 0..3, sits at
 *   1024 + lane * 16 + jj * 4 and belongs to step j = 4 (t / 2) + jj: bits 0-15 are the two
 *   index bytes of row 16 tile + g for the step's first (t even) or last (t odd) 16 columns,
 *   bits 16-31 the same for row 16 tile + g + 8.  Words are little-endian.
 */
#define SLIM_LAYOUT_DECODE_TILED 1

/* Bytes of the tiled copy (ceil(d_out / 64) * 64 * d_in * 3 / 8), or 0 when the layout cannot hold the shape. */
size_t slim_tiled_bytes(int d_out, int d_in, int layout_id);

/*
 * vals / meta as produced by slim_pack -> tiled_out (slim_tiled_bytes bytes, device, 16-byte
 * aligned).  Integer-only and bit-exact; done once per layer.
 */
slim_status_t slim_repack_tiled(const uint8_t* vals, const uint8_t* meta, int d_out, int d_in, int layout_id,
                                void* tiled_out, void* cuda_stream);

/*
 * The layer forward of slim_linear_fwd (same equation, same rounding, same workspace rules) for
 * 1 <= b <= 16 on a decode-tiled weight.  One kernel launch streams the weight, R and L exactly
 * once.  Needs d_in % 256 == 0, d_out % 16 == 0, r % 16 == 0, r <= 3072; other problems return
 * SLIM_ERR_UNSUPPORTED_SHAPE (use slim_linear_fwd on the packed weight).
 */
slim_status_t slim_linear_fwd_tiled(const void* X, int b, const void* tiled, int layout_id, float s, const void* L,
                                    const void* R, int r, int d_out, int d_in, void* Y, void* workspace,
                                    size_t workspace_bytes, uint32_t* status_dev, void* cuda_stream);

/*
 * Which copy of a weight serves small-batch calls of this shape faster on the current device:
 * 0 = the packed format (slim_linear_fwd), SLIM_LAYOUT_DECODE_TILED = the decode-tiled copy
 * (slim_linear_fwd_tiled).  The tiled kernel streams large weights at a higher rate but has a
 * longer fixed start and end that grows with the batch (activations and T are staged by few warps):
 * the rule is "tiled when the packed weight has 64 MiB or more and b <= 4 (b <= 2 when d_out < d_in)",
 * from timings of both
 * kernels on the LLaMA-2 layer shapes.  Returns 0 as well for shapes the tiled kernel does not take
 * and for illegal arguments.  (Storage layout is the implementation's choice: Sec. 4 "Speedup"
 * measures the layer, the paper fixes no format.)
 */
int slim_decode_layout_hint(int b, int d_out, int d_in, int r);

/* Host-buffer form of slim_linear_fwd_tiled (see slim_linear_fwd_host). */
slim_status_t slim_linear_fwd_tiled_host(const void* X_host, int b, const void* tiled, int layout_id, float s,
                                         const void* L, const void* R, int r, int d_out, int d_in, void* Y_host,
                                         void* x_dev, void* y_dev, void* workspace, size_t workspace_bytes,
                                         uint32_t* status_dev, void* cuda_stream);

/*
 * Host-buffer form of the same operation, for callers whose activations live
 * in host memory: X_host and Y_host are HOST pointers (pinned memory gives
 * asynchronous copies; no alignment rule); the packed weight, the adapters and
 * the workspace stay DEVICE pointers (weights are resident, activations
 * travel).  Copies X in, runs slim_linear_fwd, copies Y out, all on
 * `cuda_stream`, and synchronises that stream before returning.  x_dev / y_dev
 * are caller-owned device staging buffers of b*d_in and b*d_out bf16 elements.
 */
slim_status_t slim_linear_fwd_host(const void* X_host, int b, const uint8_t* vals,
                                   const uint8_t* meta, float s, const void* L, const void* R,
                                   int r, int d_out, int d_in, void* Y_host, void* x_dev,
                                   void* y_dev, void* workspace, size_t workspace_bytes,
                                   uint32_t* status_dev, void* cuda_stream);

/*
 * SLiM-Quant: the scale of a weight matrix and its 4-bit codes (Sec. 3.1 "SLiM-Quant Quantization
 * Method", Eq. 2-7, Algorithm 1; bins: App. "Settings and Hyperparameters").  The step before
 * slim_pack: W[d_out][d_in] float32 in, dense int8 codes in [-8, 7] and the scale s out.
 *   histogram of |W| over [0, M], M = max |W|, B = max(512, min(d_in d_out / 1000, 20000)) uniform bins,
 *     a bin standing for its centre x_i with weight count_i / N;
 *   E(alpha) = sum_{x_i <= alpha} p_i (alpha / 8 * round(8 x_i / alpha) - x_i)^2 + sum_{x_i > alpha} p_i (alpha - x_i)^2;
 *   candidates alpha = k M / 10, k = 1..10, then alpha_low - M/10 + j M/100, j = 1..19, capped at M, around
 *     the best coarse one; alpha* = the first minimiser (ties: the smaller alpha);
 *   code = clamp(rint(8 W / alpha*), -8, 7), s = alpha* / 8.
 * Decisions are taken in fixed precision so that the result is reproducible bit for bit: the bin of a
 * weight is min(B - 1, (int)((|w| / M) * B)) in binary32; E in binary64, bins added in ascending order,
 * every operation rounded on its own; codes rint((w / alpha32) * 8) in binary32.
 * scale_alpha (DEVICE, 2 floats): [0] = s, [1] = alpha*.  The workspace (slim_quant_workspace_bytes,
 * DEVICE, 16-byte aligned) also receives, after the histogram, the table of the 29 (alpha, E) pairs
 * tried (float64 pairs, coarse then fine; a fine candidate that is not positive is listed with the
 * best error so far plus one) followed by alpha* as float64: at byte offset 256 + round_up(4 B, 256).
 * A NaN or infinity in W sets the SLIM_ERR_INVALID_ARG bit of *status_dev and gives scale 0; an
 * all-zero W gives scale 0 and codes 0.  Four launches on the stream; nothing is synchronised.
 */
size_t slim_quant_workspace_bytes(int d_out, int d_in);
slim_status_t slim_quant(const float* W, int d_out, int d_in, int8_t* codes, float* scale_alpha, void* workspace,
                         size_t workspace_bytes, uint32_t* status_dev, void* cuda_stream);

/*
 * The 2:4 mask of the pipeline's second step (Sec. 3 and Fig. 1: the quantized weights are sparsified by a
 * one-shot pruning method; metric of Sec. 3.2: the product of the magnitudes of weight and input).
 * In every aligned group of four along d_in the two entries with the largest |codes[n][k]| * xbar[k]
 * are kept (mask 1), equal metrics go to the lower index; xbar NULL: magnitude pruning.  The metric is
 * one binary32 multiplication, so the mask is reproducible bit for bit.  codes [d_out][d_in] int8,
 * xbar [d_in] float32 (average input magnitude per channel: non-negative and finite, else the
 * SLIM_ERR_INVALID_ARG bit of *status_dev is set), mask [d_out][d_in] uint8; d_in % 4 == 0; DEVICE
 * pointers, 16-byte aligned.  The output is slim_pack's `mask` argument.
 */
slim_status_t slim_mask_top2(const int8_t* codes, const float* xbar, int d_out, int d_in, uint8_t* mask, uint32_t* status_dev,
                             void* cuda_stream);

/*
 * Quantized adapters (Sec. 3.3 "Low-rank Adapter Quantization": 4-bit AbsMax group quantization,
 * groups of 128 elements share one quantization parameter; grid of Sec. 3.1 Eq. 2 / Eq. 5).
 * An adapter is a row-major bf16 matrix A[rows][cols] whose rows run along the contraction axis
 * of its product (R[r][d_in]; L[d_out][r]); a group is 128 consecutive elements of a row (the last
 * group of a row may be shorter).  Storage, 4.125 bits per element:
 *   codes[rows][cols / 2]             two int4 codes per byte, even column in the low nibble;
 *   scales[rows][ceil(cols / 128)]    bf16, scale = absmax / 7 (binary32 division, nearest-even).
 * code = clamp(rint(a / scale), -8, 7), division in binary32, ties to even; a group of zeros has
 * scale 0 and codes 0; the value of an element is code * scale.  cols must be even; all pointers
 * are DEVICE pointers, 16-byte aligned.  (Magnitudes below the smallest normal binary32 number are
 * handled as the device's flush-to-zero arithmetic handles them.)
 */
size_t slim_adapter_code_bytes(int rows, int cols);     /* 0 for illegal arguments */
size_t slim_adapter_scale_bytes(int rows, int cols);
/* Quantize: bit-exact with the definition above. */
slim_status_t slim_pack_adapter(const void* A, int rows, int cols, uint8_t* codes, void* scales, void* cuda_stream);
/* The bf16 matrix nearest to the values the codes and scales stand for. */
slim_status_t slim_unpack_adapter(const uint8_t* codes, const void* scales, int rows, int cols, void* A_out,
                                  void* cuda_stream);

/*
 * The layer forward with quantized adapters (SLiM-LoRA^Q; Sec. 3.3, with the layer of Sec. 3.2):
 * slim_linear_fwd with L and R given as codes and scales (Lq/Ls for L[d_out][r], Rq/Rs for
 * R[r][d_in]).  r >= 16.  For b <= 16 and shapes the decode kernel takes, the decode kernel reads codes
 * and scales as they are (through tensor maps; L's codes with plain loads when their rows of r / 2 bytes
 * are no 16-byte multiples): it multiplies the exact integer codes and scales its accumulator once
 * per group, and a call moves
 * 4.125 bits per adapter element instead of 16 (Sec. 4 "Speedup": quantized adapters cut the
 * adapters' share of the layer's time).  Otherwise the adapters are expanded to bf16 (each value
 * rounded once, nearest even) into the tail of the workspace and the kernel slim_linear_fwd would
 * pick runs on them: what is saved then is the resident size of the adapters only.  The workspace
 * must have slim_workspace_bytes_q bytes (its first slim_workspace_bytes bytes are the ordinary
 * workspace, prepared by slim_workspace_reset as usual).
 */
size_t slim_workspace_bytes_q(int b, int d_out, int d_in, int r);
slim_status_t slim_linear_fwd_q(const void* X, int b, const uint8_t* vals, const uint8_t* meta, float s,
                                const uint8_t* Lq, const void* Ls, const uint8_t* Rq, const void* Rs, int r,
                                int d_out, int d_in, void* Y, void* workspace, size_t workspace_bytes,
                                uint32_t* status_dev, void* cuda_stream);

/*
 * Small-batch forward that allocates nothing.  (The paper has no counterpart:
 * this entry point exists for the deployment constraint described here.)
 *
 * Some hosts of this library must not call cudaMalloc while they run: a serving
 * loop that cannot afford the device-wide synchronisation an allocation causes,
 * a plug-in living inside a runtime that has handed all device memory to its
 * own pool, a process working under a fixed memory budget.  Such a caller
 * cannot provide the workspace slim_linear_fwd asks for, so this variant keeps
 * the decode kernel's scratch (split-K partial sums and barrier counters) in a
 * fixed array of SLIM_NOALLOC_SCRATCH_BYTES inside the library's device image.
 * Every GPU that loads the library holds that array until the process exits.
 *
 * Same operation, arguments and rounding as slim_linear_fwd, for b <= 16 and the
 * shapes the decode kernel takes (d_in % 256 == 0); other problems return
 * SLIM_ERR_UNSUPPORTED_SHAPE, and a problem whose scratch would exceed the
 * array returns SLIM_ERR_WORKSPACE (all LLaMA-2 7B/13B/70B layer shapes fit).
 * The call makes no cudaMalloc / cudaFree and uses no allocating library
 * routine; inputs and outputs are still the caller's device buffers.
 *
 * The first call on a device looks up the array's device address (the device
 * must be current); make that first call before starting any stream capture.
 * All calls on a device share the one array, which keeps the previous call's
 * contents (the part a call uses is re-initialised on the stream at its start):
 * two calls that overlap on the GPU - different streams, no ordering between
 * them - race on it and produce garbage.  Issue them on one stream or order
 * them with events.
 */
#define SLIM_NOALLOC_SCRATCH_BYTES (16u << 20)
slim_status_t slim_linear_fwd_noalloc(const void* X, int b, const uint8_t* vals, const uint8_t* meta,
                                      float s, const void* L, const void* R, int r, int d_out,
                                      int d_in, void* Y, uint32_t* status_dev, void* cuda_stream);

/*
 * Bytes of the built-in array slim_linear_fwd_noalloc would use for this problem (host-side
 * arithmetic, no device needed); 0 when the entry point does not take the problem at all.  A
 * value above SLIM_NOALLOC_SCRATCH_BYTES means the call would return SLIM_ERR_WORKSPACE.
 */
size_t slim_noalloc_scratch_needed(int b, int d_out, int d_in, int r);

/* The kernel family slim_linear_fwd would pick for this problem. */
slim_kernel_t slim_select_kernel(int b, int d_out, int d_in, int r);

/* Number of kernels the last slim_linear_fwd* call on this host thread launched. */
int slim_last_launch_count(void);

/*
 * Token-tile width (64 or 256 tokens) of the prefill kernel the last slim_linear_fwd* call on this host
 * thread launched, 0 if that call ran another kernel.  The prefill kernel has a wide variant for problems
 * with enough 128-row x 256-token tiles for a quarter of the SMs or more and a narrow one for the rest; tests use this query to
 * make sure they exercise the variant they mean to.
 */
int slim_last_token_tile(void);

const char* slim_strerror(slim_status_t status);
const char* slim_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SLIM_H */
