/*
 * mxq.h -- C-ABI of libmxq: block-wise microscaled FP4 (E2M1) quantization of whole tensors with
 * per-block scale selection, scored by per-block SSE and per-tensor MSE, on one NVIDIA B200
 * (sm_100a).  Implements the quantization recipes studied in "Finer is Better (with the Right
 * Scaling)": MX power-of-two scales (Eq. 1), abs-max rounded to an FP8 scale format (Eq. 2), the
 * prevent-zero clamp (Eq. 3), 4-over-6 (Eq. 4), hierarchical tensor + block scaling and the
 * brute-force search over every scale code (Experimental Setup).
 *
 * Conventions for every entry point
 *   - Pointers named d_* or documented "device" are DEVICE pointers owned by the caller.  The
 *     library never allocates, frees or keeps them.  All device buffers must be 16-byte aligned.
 *   - Calls validate their arguments on the host, enqueue kernels on `cuda_stream` (a
 *     cudaStream_t passed as void*; NULL = the default stream) and return without synchronising.
 *     Nothing is launched when validation fails.
 *   - Return value: MXQ_OK (0) or a positive mxq_status.  Nothing throws, aborts or prints.
 *   - Results are deterministic from run to run (no floating-point atomics).
 *   - Inputs must be finite.  NaN or Inf elements give unspecified (but memory-safe) outputs.
 *   - Threads.  Entry points may be called from several host threads at once (on the same or on
 *     different devices and streams): the library keeps no per-call host state, its first-use caches
 *     (SM count, resident CTAs per kernel) are atomics whose racing writers store equal values, and
 *     mxq_last_cuda_error() is per thread.  Two things are process-wide and therefore shared by all
 *     threads: the options of mxq_set_option() (a call reads the option once, when it is made; changing
 *     it while another thread is inside mxq_quantize_ex affects only calls made afterwards), and the
 *     scratch array of mxq_tensor_mse_static() (see there).  As with any CUDA library, the device that
 *     owns the pointers must be the calling thread's current device.
 *
 * Data layout
 *   x            n elements, contiguous; a block is B consecutive elements of the flat array
 *                (a row-major matrix whose row length is a multiple of B is blocked along rows).
 *   out_codes    n/2 bytes; byte j holds element 2j in bits 0..3 and element 2j+1 in bits 4..7;
 *                a 4-bit code is sign<<3 | index into {0, 0.5, 1, 1.5, 2, 3, 4, 6}
 *                (Experimental Setup, FP4 value set); the sign bit is the sign bit of the input.
 *   out_scales   n/B bytes, one scale code per block in the chosen scale format.
 *   out_block_sse n/B floats: sum over the block of (x - dequantized x)^2, accumulated in
 *                binary32 in element order with fused multiply-adds; may be NULL.
 */
#ifndef MXQ_H_
#define MXQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MXQ_OK = 0,
    MXQ_ERR_NULL = 1,      /* a required pointer is NULL */
    MXQ_ERR_BAD_ENUM = 2,  /* dtype, scale_fmt or recipe out of range */
    MXQ_ERR_BAD_SHAPE = 3, /* n == 0, n not a multiple of block_size, block_size not in {2,4,8,16,32,64},
                              or n so small that n/2 is not an integer */
    MXQ_ERR_ALIGN = 4,     /* a device pointer is not 16-byte aligned */
    MXQ_ERR_BAD_SCALE = 5, /* global_scale is not finite or is <= 0 */
    MXQ_ERR_WORKSPACE = 6, /* workspace NULL or smaller than required */
    MXQ_ERR_CUDA = 7,      /* a CUDA call failed; see mxq_last_cuda_error() */
    MXQ_ERR_TOO_LARGE = 8  /* the size exceeds the fixed capacity of an entry point that owns its scratch */
} mxq_status;

typedef enum { MXQ_F32 = 0, MXQ_BF16 = 1 } mxq_dtype;

/* Block-scale formats (Background).  UE8M0: 2^(code-127), codes 0..254.  UE4M3: E4M3 with the
 * sign bit unused, bias 7, subnormals, smallest nonzero 2^-9, largest 448, codes 0..0x7E.
 * UE5M3: 5 exponent + 3 mantissa bits, bias 15, subnormals, smallest nonzero 2^-17, largest
 * 1.75*2^16, codes 0..0xFE (the paper names this format without defining it; this is the
 * library's definition). */
typedef enum { MXQ_SF_UE8M0 = 0, MXQ_SF_UE4M3 = 1, MXQ_SF_UE5M3 = 2 } mxq_scale_fmt;

/* Scale-selection recipes (Experimental Setup).
 *   ABSMAX     Eq. 2 with M = 6: code = Round_SF(amax / g / 6), round-to-nearest-even, clipped to
 *              the largest finite code.  With MXQ_SF_UE8M0 the rule is Eq. 1 instead: the
 *              largest power of two <= amax / g / 6.
 *   *_PZ       Eq. 3: a scale that rounds to zero is replaced by the smallest nonzero scale
 *              (code 1).  No effect for UE8M0, whose codes are all nonzero.
 *   4O6        Eq. 4: candidates Round_SF(amax/g/6) and Round_SF(amax/g/4); the block is
 *              quantized with both and the one with the smaller SSE is kept (tie: M = 6).
 *   BRUTE      every finite scale code is tried (BRUTE_PZ: every code with a nonzero value);
 *              smallest SSE wins, equal SSE keeps the smaller code.  A code whose decode scale
 *              S*g is not a finite float is skipped.
 *   ABSMAX_OCP MXQ_SF_UE8M0 only: the power-of-two rule as the OCP MX specification words it (the
 *              Background paraphrases it; Eq. 1 as printed differs): scale exponent = exponent of the
 *              block maximum minus the exponent of the largest FP4 value, S = 2^(floor(log2(amax/g)) - 2).
 *              The maximum lands in [4, 8) and is clipped above 6; S is the scale of Eq. 1 or twice it.
 *   ABSMAX_CLIP7 MXQ_SF_UE8M0 only: the power-of-two scale that maps the block maximum into [3.5, 7)
 *              (the clipping recipe of a cited work that the Background describes):
 *              S = 2^floor(log2(amax/g / 3.5)); a maximum that lands in (6, 7) is clipped to 6.
 *              S is the scale of Eq. 1 or twice it.
 * Hierarchical scaling is any recipe called with global_scale != 1. */
typedef enum {
    MXQ_ABSMAX = 0, MXQ_ABSMAX_PZ = 1, MXQ_4O6 = 2, MXQ_4O6_PZ = 3, MXQ_BRUTE = 4, MXQ_BRUTE_PZ = 5,
    MXQ_ABSMAX_OCP = 6, MXQ_ABSMAX_CLIP7 = 7
} mxq_recipe;

/*
 * mxq_quantize -- quantize a float32 tensor on the default stream (Experimental Setup: Eq. 2-4,
 * "quant(v_i / S)", hierarchical scaling, brute-force search).
 *   x             device, n floats.
 *   n             element count, a positive multiple of block_size.
 *   block_size    2, 4, 8, 16, 32 or 64.
 *   scale_fmt     mxq_scale_fmt.         recipe   mxq_recipe.
 *   global_scale  g > 0, finite: the per-tensor decode scale of hierarchical scaling; 1 = none.
 *                 Block targets are found from amax/g; elements are divided by D = fl32(S*g).
 *   out_codes, out_scales, out_block_sse   device outputs as described above (sse may be NULL).
 * Per element: t = fl32(x / D), code = sign | RNE_E2M1(min(|t|, 6)); D = 0 gives magnitude 0.
 */
int mxq_quantize(const float* x, size_t n, int block_size, int scale_fmt, int recipe, float global_scale,
                 uint8_t* out_codes, uint8_t* out_scales, float* out_block_sse);

/*
 * mxq_quantize_ex -- as mxq_quantize, with an input dtype, an optional device-resident global
 * scale and a stream.
 *   x               device, n elements of `dtype` (MXQ_F32 or MXQ_BF16; bf16 is widened exactly).
 *   d_global_scale  device pointer to one float holding g, or NULL.  When non-NULL it overrides
 *                   `global_scale` and is read by the kernel at run time (no host
 *                   synchronisation); it must hold a finite positive value when the kernel runs.
 */
int mxq_quantize_ex(const void* x, int dtype, size_t n, int block_size, int scale_fmt, int recipe,
                    float global_scale, const float* d_global_scale, uint8_t* out_codes, uint8_t* out_scales,
                    float* out_block_sse, void* cuda_stream);

/*
 * mxq_quantize_batch -- mxq_quantize_ex over a LIST of tensors in one launch: the weight matrices of a
 * model, say, which the experiments of the paper quantize one recipe at a time (Results, downstream
 * evaluation: every MLP weight matrix).  One persistent grid walks all tensors, so the launch overhead,
 * the ramp at the start and the drain at the end are paid once for the whole list instead of once per
 * tensor.  Outputs are those of mxq_quantize_ex on each tensor, bit for bit.
 *   h_descs     HOST array of n_tensors descriptors (read during the call: validation, grid size).
 *   d_descs     DEVICE copy of the same array, made by the caller (it owns the memory; the kernel reads it,
 *               so it must stay unchanged until the launch has run).  16-byte aligned.
 *   n_tensors   1 .. 1024 (MXQ_ERR_TOO_LARGE beyond).
 *   dtype, block_size, scale_fmt, global_scale, d_global_scale   common to all tensors, as for mxq_quantize_ex.
 *   recipe      any recipe except the brute-force ones (their launches last milliseconds; MXQ_ERR_BAD_ENUM).
 * Every tensor: x, out_codes, out_scales non-NULL, out_block_sse optional, all 16-byte aligned; n a
 * positive multiple of 64 (MXQ_ERR_BAD_SHAPE otherwise).
 */
typedef struct {
    const void* x;        /* device, n elements of the call's dtype */
    uint8_t* out_codes;   /* device, n / 2 bytes */
    uint8_t* out_scales;  /* device, n / block_size bytes */
    float* out_block_sse; /* device, n / block_size floats, or NULL */
    size_t n;             /* element count */
} mxq_tensor_desc;
int mxq_quantize_batch(const mxq_tensor_desc* h_descs, const mxq_tensor_desc* d_descs, size_t n_tensors, int dtype,
                       int block_size, int scale_fmt, int recipe, float global_scale, const float* d_global_scale,
                       void* cuda_stream);

/*
 * mxq_fake_quantize -- quantize and de-quantize in one pass: out_i = fl32(grid(code_i) * D_b), the
 * values a model computes with when its MLP weights or activations are held in this format (the
 * setting of the downstream experiments in Results).  Bit-identical to mxq_quantize_ex followed by mxq_dequantize, without writing
 * codes, scales or SSE.
 *   x, dtype, n, block_size, scale_fmt, global_scale, d_global_scale, cuda_stream   as for mxq_quantize_ex.
 *   recipe     any recipe except the brute-force ones (MXQ_ERR_BAD_ENUM for those: run mxq_quantize_ex
 *              and mxq_dequantize instead).
 *   d_out      device, n elements of out_dtype (MXQ_F32, or MXQ_BF16 = the binary32 value rounded to
 *              bf16, round-to-nearest-even); may not alias x.
 */
int mxq_fake_quantize(const void* x, int dtype, size_t n, int block_size, int scale_fmt, int recipe,
                      float global_scale, const float* d_global_scale, void* d_out, int out_dtype, void* cuda_stream);

/*
 * mxq_tensor_amax -- first stage of hierarchical scaling (Experimental Setup): the largest magnitude
 * of the whole tensor, from which the per-tensor scale is derived.
 *   d_out_amax  device, one float: max_i |x_i| (0 for an all-zero tensor).
 *   d_out_global_scale  device, one float, or NULL: receives g = amax / (6*448) computed in
 *               binary32 (1 if amax == 0), ready to be passed as d_global_scale.
 */
int mxq_tensor_amax(const void* x, int dtype, size_t n, float* d_out_amax, float* d_out_global_scale,
                    void* cuda_stream);

/* Host helper: the same g = amax / 2688 in binary32 (1 if amax is 0 or not finite). */
float mxq_global_scale_from_amax(float amax);

/*
 * mxq_tensor_mse -- tensor MSE = (sum of the block SSEs) / n (Eq. 4 text, "MSE(v, S)"; Results,
 * numerical study), as a fixed-shape two-level tree in binary64: the same inputs always give the
 * same bits.
 *   d_block_sse     device, n_blocks floats.
 *   n               element count the SSEs cover (the divisor).
 *   d_out_mse       device, one double.
 *   d_workspace     device scratch of at least mxq_tensor_mse_workspace_bytes(n_blocks) bytes;
 *                   contents are overwritten; no need to clear it.
 */
size_t mxq_tensor_mse_workspace_bytes(size_t n_blocks);
int mxq_tensor_mse(const float* d_block_sse, size_t n_blocks, size_t n, double* d_out_mse, void* d_workspace,
                   size_t workspace_bytes, void* cuda_stream);

/*
 * mxq_quantize_mse -- mxq_quantize_ex and the tensor MSE of its result in one call (Eq. 4 text, "MSE(v, S)";
 * Results, numerical study: every quantization is scored by its MSE).  The quantization kernel adds up
 * the block SSEs it produces -- binary64, a fixed order per thread, a fixed tree per CTA -- and a one-CTA
 * kernel adds the per-CTA sums with the second level of mxq_tensor_mse's tree and divides by n: the
 * block SSEs are not read back from memory, and out_block_sse may be NULL when only the MSE is wanted.
 *   x .. out_block_sse, cuda_stream   as for mxq_quantize_ex (every recipe, brute force included).
 *   d_out_mse     device, one double: (sum of all block SSEs) / n.
 *   d_workspace   device scratch of at least mxq_tensor_mse_workspace_bytes(n / block_size) bytes;
 *                 contents are overwritten; no need to clear it.
 * Codes, scale bytes and block SSEs are those of mxq_quantize_ex bit for bit.  The MSE is deterministic
 * (same device, same arguments: same bits) and agrees with mxq_tensor_mse on the same SSEs to within the
 * rounding of binary64 sums taken in a different order (about 1e-15 relative).
 */
int mxq_quantize_mse(const void* x, int dtype, size_t n, int block_size, int scale_fmt, int recipe,
                     float global_scale, const float* d_global_scale, uint8_t* out_codes, uint8_t* out_scales,
                     float* out_block_sse, double* d_out_mse, void* d_workspace, size_t workspace_bytes,
                     void* cuda_stream);

/*
 * mxq_tensor_mse_static -- mxq_tensor_mse for callers that have no device memory to lend as a
 * workspace and must not allocate any: for example a plug-in or operator that a serving runtime
 * hands nothing but its input and output buffers, while the runtime's own pool has already
 * reserved the rest of the GPU (a raw cudaMalloc there fails, or stalls the device while it
 * synchronises), or a latency-bound loop in which an allocation is not acceptable.  The paper has
 * no counterpart of this call; it computes exactly what mxq_tensor_mse computes (same kernels,
 * same tree, same bits) and differs only in where the 1024 first-level partial sums live: in an
 * 8 KiB array that is part of the library image, present on every GPU that loads the library
 * until the process exits.  The call allocates nothing and frees nothing.
 *   d_block_sse, n_blocks, n, d_out_mse, cuda_stream   as for mxq_tensor_mse (caller-owned).
 *   n_blocks    at most MXQ_TENSOR_MSE_STATIC_MAX_BLOCKS; a larger count returns
 *               MXQ_ERR_TOO_LARGE and launches nothing (use mxq_tensor_mse with a workspace).
 * The first call on each device looks up the array's device address (the device must be current,
 * as for every call); make that first call outside any stream capture.  All calls on a device
 * share the one array and each overwrites what the previous one left; nothing needs clearing
 * between calls.  Two calls whose kernels can overlap on the GPU (different streams, no ordering
 * between them) race on the array and give undefined results: keep such calls on one stream or
 * order them with events.
 */
#define MXQ_TENSOR_MSE_STATIC_MAX_BLOCKS ((size_t)1 << 31)
int mxq_tensor_mse_static(const float* d_block_sse, size_t n_blocks, size_t n, double* d_out_mse, void* cuda_stream);

/*
 * mxq_dequantize -- de-quantization, a multiplication by the scale (Experimental Setup):
 * out_i = fl32(grid(code_i) * D_b), D_b = fl32(S_b * g); MXQ_BF16 output rounds that to bf16 (RNE).
 *   d_codes  n/2 bytes;  d_scales  n/block_size bytes;  d_out  n elements of out_dtype.
 * A scale byte that is not a finite code of the format decodes as NaN.
 */
int mxq_dequantize(const uint8_t* d_codes, const uint8_t* d_scales, size_t n, int block_size, int scale_fmt,
                   float global_scale, void* d_out, int out_dtype, void* cuda_stream);

/*
 * mxq_dequantize_ex -- mxq_dequantize with an optional device-resident tensor scale, so that the
 * hierarchical flow (mxq_tensor_amax -> g on the device -> mxq_quantize_ex -> ... -> de-quantize) never
 * has to read g back to the host (Experimental Setup, hierarchical scaling).
 *   d_global_scale  device pointer to one float holding g, or NULL.  When non-NULL it overrides
 *                   `global_scale` (which is then not checked) and is read by the kernel at run time.
 */
int mxq_dequantize_ex(const uint8_t* d_codes, const uint8_t* d_scales, size_t n, int block_size, int scale_fmt,
                      float global_scale, const float* d_global_scale, void* d_out, int out_dtype, void* cuda_stream);

/*
 * mxq_block_clip_sse -- the clipping part of the block SSE (Appendix, "Clipping only MSE": the MSE
 * plots of the numerical study restricted to their clipping portion).  For every block, the sum
 * of (x - x_hat)^2 over the elements whose scaled magnitude exceeds the largest FP4 value,
 * |fl32(x / D)| > 6 with D = fl32(S * g) -- they are all mapped to +-6 -- accumulated like the block
 * SSE (binary32, element order, fused multiply-adds).  A zero decode scale clips nothing.
 *   x, dtype, n, block_size, scale_fmt, global_scale, d_global_scale   as for mxq_quantize_ex.
 *   d_scales      device, n/block_size scale codes as written by the quantizer.
 *   out_clip_sse  device, n/block_size floats (NaN for a byte that is not a code of the format).
 * Dividing the sum of these values by n gives the clipping-only MSE of the tensor.
 */
int mxq_block_clip_sse(const void* x, int dtype, size_t n, int block_size, int scale_fmt, float global_scale,
                       const float* d_global_scale, const uint8_t* d_scales, float* out_clip_sse, void* cuda_stream);

/*
 * mxq_histograms -- bin utilisation of a quantized tensor (Appendix, histograms of entries and of
 * scaling factors per recipe).
 *   d_codes, d_scales   device, outputs of the quantizer for n elements in blocks of block_size.
 *   d_code_hist   device, 16 unsigned 64-bit counters: occurrences of each 4-bit code (sign<<3 | index).
 *   d_scale_hist  device, 256 unsigned 64-bit counters: occurrences of each scale code.
 * Counts are ADDED to both arrays (clear them first for a fresh histogram; several tensors may be
 * accumulated).  Integer sums: the result does not depend on the order of execution.
 */
int mxq_histograms(const uint8_t* d_codes, const uint8_t* d_scales, size_t n, int block_size,
                   unsigned long long* d_code_hist, unsigned long long* d_scale_hist, void* cuda_stream);

/*
 * mxq_segment_mse -- MSE of consecutive, equally long segments of a tensor in one launch (Results,
 * numerical study: one segment per standard deviation sigma, 50,000 blocks each).
 *   d_block_sse          device, n_blocks floats (or clipping SSEs).
 *   blocks_per_segment   n_blocks must be a multiple of it.
 *   elems_per_segment    the divisor (blocks_per_segment * block size).
 *   d_out_mse            device, n_blocks / blocks_per_segment doubles.
 * Fixed-shape binary64 tree per segment: the same inputs always give the same bits.  Needs no
 * workspace.
 */
int mxq_segment_mse(const float* d_block_sse, size_t n_blocks, size_t blocks_per_segment, size_t elems_per_segment,
                    double* d_out_mse, void* cuda_stream);

/*
 * mxq_mask_interval -- the pre-quantization diagnostic of the appendix (entries whose magnitude lies
 * in a chosen interval are zeroed at full precision): out_i = 0 when lo <= |x_i| < hi, else x_i.
 *   x, d_out   device, n elements of dtype (MXQ_F32 or MXQ_BF16); d_out may be x (in place).
 *   lo, hi     0 <= lo <= hi, else MXQ_ERR_BAD_SCALE.  NaN entries pass unchanged.
 */
int mxq_mask_interval(const void* x, int dtype, size_t n, float lo, float hi, void* d_out, void* cuda_stream);

/* Process-wide options, read by the entry points when they are called.
 *
 * MXQ_OPT_BRUTE_PRUNE (default 0).  With 0 the brute-force recipes evaluate every finite scale code
 * on every block, exactly as the search is stated (Experimental Setup).  With 1 a warp of the kernel
 * leaves out the codes that provably cannot change an output of any block it holds:
 *   - decode scales of at least four times the largest magnitude: every element quantizes to zero
 *     (|v|/D <= 1/4 rounds to the grid value 0), so all of them have the SSE of the all-zero
 *     quantization, which is entered once with the smallest such code;
 *   - decode scales so large that the elements they send to zero alone already cost more than the
 *     best SSE found so far, in every block;
 *   - decode scales so small that the saturation error of the largest element alone already exceeds
 *     the best SSE found so far, in every block.
 * The bounds are evaluated in the kernel's own binary32 arithmetic and compared strictly, so the
 * outputs (codes, scale bytes, block SSE; ties to the smaller code) are bit-identical to the full
 * sweep; only the time differs, by an amount that depends on the data.  For block sizes up to 16
 * the kernel first sorts the blocks of each CTA by magnitude (in shared memory), so that a warp holds
 * blocks of like size and its bounds are tight.  The paper states no such shortcut.
 *
 * mxq_set_option: MXQ_ERR_BAD_ENUM for an unknown option or a value outside {0, 1}.
 * mxq_get_option: MXQ_ERR_NULL for a NULL out_value (host pointer). */
enum { MXQ_OPT_BRUTE_PRUNE = 1 };
int mxq_set_option(int option, int value);
int mxq_get_option(int option, int* out_value);

/* Number of kernels the library has launched in this process (all entry points), for
 * accounting in benchmarks. */
unsigned long long mxq_launch_count(void);

const char* mxq_status_string(int status);
/* The cudaError_t (as int) behind the most recent MXQ_ERR_CUDA on this thread, else 0. */
int mxq_last_cuda_error(void);
/* major*10000 + minor*100 + patch */
int mxq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MXQ_H_ */
