/*
 * libthc -- the data-parallel hot path of Tensor Homomorphic Compression (THC,
 * arxiv 2302.08545) as hand-written CUDA for sm_100a, behind a C ABI.
 *
 * One round, as the paper states it (Algorithm 3, the coloured THC lines):
 *     thc_prepare     preliminary stage: per RHT block, M = t_p * max_i ||x_i|| / sqrt(B)
 *     thc_compress    RHT -> truncate -> stochastic quantisation to b-bit table indices -> pack
 *     thc_aggregate   the parameter server's only job: Y = sum_i T[Z_i], in integers
 *     thc_decompress  Y/n -> real values -> inverse RHT
 * and around them: thc_prepare_compress (the first two in one launch), thc_prepare_minmax (the
 * exact range of Algorithm 1's preliminary stage instead of the norm-based one),
 * thc_quantize_rotated, thc_error_feedback / thc_accumulate_error (Algorithm 3's residual),
 * thc_aggregate_decompress (the last two in one launch, for a caller that holds every
 * worker's indices on one GPU).
 *
 * Conventions shared by every call
 *   - "device" pointers are CUDA device addresses on the device that was current when the
 *     context was created; "host" pointers are ordinary host memory.
 *   - Arrays of per-worker pointers (grads, packed, rotated) are HOST arrays holding DEVICE
 *     pointers; the library copies them into kernel arguments, so they may be freed or
 *     reused as soon as the call returns.
 *   - Every device buffer is owned by the caller.  Device buffers must be 16-byte aligned.
 *     The library owns only the context (a few hundred bytes of device memory for the
 *     status word and scheduling counters, allocated by thc_create).
 *   - The round calls (and thc_quantize_rotated, thc_prepare_compress, thc_prepare_minmax,
 *     thc_error_feedback, thc_accumulate_error) only enqueue work on `stream`
 *     (a cudaStream_t passed as void*; NULL = the legacy default stream) and return without
 *     synchronising.  They allocate nothing.  Calls that share a context must be issued
 *     on one stream (or be ordered by the caller): they share the context's counters.
 *     Different contexts are independent: they may be used from different host threads and
 *     on different streams at the same time.
 *   - Return value: THC_OK or a negative THC_E* code; thc_strerror() gives text, and for
 *     THC_ECUDA the text of the CUDA error last seen by this thread's library calls.
 *   - Conditions met on the device never trap: they set bits that thc_status() reports.
 *
 * Layouts (coordinate j = 0 .. d_pad-1, d_pad = d rounded up to a multiple of B = 2^k)
 *   gradient   d elements, fp32 or bf16, contiguous; coordinates d..d_pad-1 count as zero
 *   scales     one fp32 M per block, nblocks = d_pad / B entries (THC_RANGE_MINMAX contexts:
 *              nblocks minima followed by nblocks maxima; thc_sizes_t.scales_count)
 *   packed     d_pad*b/8 bytes per worker; index j in bits [j*b, j*b + b) of the little-endian bit
 *              stream, i.e. bits [(j mod 8/b)*b, +b) of byte j*b/8 where b divides 8
 *   sum        d_pad little-endian unsigned integers of acc_bits bits
 *   rotated    d_pad fp32 per worker: the RHT output before truncation (optional)
 *   out        d fp32
 */
#ifndef THC_H_
#define THC_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define THC_OK             0
#define THC_EINVAL        (-1)  /* bad configuration or argument (null, misaligned, n = 0, ...) */
#define THC_EUNSUPPORTED  (-2)  /* valid but not implemented (e.g. granularity > 255)           */
#define THC_ECUDA         (-3)  /* a CUDA call failed, or the context has no device             */
#define THC_EWORKSPACE    (-4)  /* workspace smaller than thc_sizes() asks for                  */

#define THC_F32   0u
#define THC_BF16  1u

#define THC_MAX_WORKERS 64u

/* thc_status() bits */
#define THC_STATUS_NONFINITE     1u  /* a block's norm was NaN/Inf: its scale was set to 0        */
#define THC_STATUS_ZERO_BLOCK    2u  /* a block had scale 0 (all-zero input): indices 0, output 0 */
                                     /* (exact range: a block whose range is [0, 0])              */
#define THC_STATUS_WAIT_TIMEOUT  4u  /* an on-device wait gave up; the call's output is invalid   */

typedef struct thc_ctx thc_ctx;   /* opaque */

/*
 * Parameters of the method (Algorithm 3, "Input" line) plus the layout choices.
 *   bits         b in {1, 2, 3, 4, 8}: bits per table index (Section 4.3)
 *   granularity  g with 2^b - 1 <= g <= 255 (Section 4.3, "granularity")
 *   table        T[0 .. 2^b - 1], 0 = T[0] < T[1] < ... < T[2^b - 1] = g (Section 4.3);
 *                the identity table with g = 2^b - 1 is Uniform THC (Section 4.2)
 *   t_p          truncation threshold Phi^-1(1 - p/2) (Section 5.2), > 0
 *   log2_block   k in [3, 22]: the RHT acts on blocks of B = 2^k coordinates (Section 5.1
 *                applied per partition)
 *   seed         shared by all workers: the diagonal D of the RHT must be common
 *   in_dtype     THC_F32 or THC_BF16 (bf16 gradients are widened exactly on load)
 *   workers      the largest number of workers thc_aggregate will sum (1..THC_MAX_WORKERS)
 *   acc_bits     width of the sums: 8, 16 or 32, or 0 = smallest with workers*g <= 2^w - 1
 *                (Section 8.4: the largest aggregate is g*n)
 */
#define THC_RANGE_NORM   0u
#define THC_RANGE_MINMAX 1u

typedef struct thc_config {
    uint32_t bits;
    uint32_t granularity;
    uint16_t table[256];
    double   t_p;
    uint32_t log2_block;
    uint64_t seed;
    uint32_t in_dtype;
    uint32_t workers;
    uint32_t acc_bits;
    uint32_t range_mode;   /* THC_RANGE_NORM (0): M = t_p max_i ||x_i|| / sqrt(B), m = -M (Section 5.3);
                              THC_RANGE_MINMAX (1): the exact minimum and maximum of the rotated
                              coordinates over all workers (Algorithm 1's preliminary stage applied
                              after the RHT): nothing is clamped; fp32 input only */
} thc_config;

typedef struct thc_sizes_t {
    uint64_t d_pad;            /* d rounded up to a multiple of the block              */
    uint64_t nblocks;          /* d_pad / B = number of scales                         */
    uint64_t packed_bytes;     /* per worker                                           */
    uint64_t sum_bytes;        /* d_pad * acc_bits / 8                                 */
    uint64_t rotated_bytes;    /* per worker, 4 * d_pad                                */
    uint64_t workspace_bytes;  /* scratch any call may need for this (d, n_local)      */
    uint32_t acc_bits;         /* the resolved accumulator width                       */
    uint32_t fused_scales;     /* 1: thc_prepare_compress is one launch for (d, n_local)  */
    uint64_t scales_count;     /* floats in `scales`: nblocks, or 2 * nblocks (minima, then
                                  maxima) in THC_RANGE_MINMAX mode                        */
} thc_sizes_t;

/* Validate `cfg` (host only) and build a context.  If a CUDA device is present, the
 * context's device block is allocated on the current device; without a device the context
 * still answers thc_sizes() and validation, and every launching call returns THC_ECUDA.
 * Launching calls must be made with that device current (THC_EINVAL otherwise).
 * Errors: THC_EINVAL (see thc_config), THC_EUNSUPPORTED, THC_ECUDA. */
int thc_create(const thc_config *cfg, thc_ctx **ctx);
int thc_destroy(thc_ctx *ctx);

/* Buffer sizes for gradients of d elements and calls that handle up to n_local workers at
 * once.  Host only. */
int thc_sizes(const thc_ctx *ctx, uint64_t d, uint32_t n_local, thc_sizes_t *sizes);

/* Preliminary stage (Section 5.3; Algorithm 3, "Send ||x_i|| / Receive ell" and
 * "M = (t_p / sqrt d) * ell"): scales[blk] = (float)(t_p * max_i ||x_i restricted to
 * block blk||_2 / sqrt(B)), norms accumulated in fp64.  A non-finite norm gives scale 0 and
 * sets THC_STATUS_NONFINITE.
 *   grads   host array of n device pointers, each d elements of cfg.in_dtype
 *   scales  device, nblocks fp32, written                                              */
int thc_prepare(thc_ctx *ctx, const void *const *grads, uint32_t n, uint64_t d,
                float *scales, void *workspace, uint64_t workspace_bytes, void *stream);

/* Worker-side compression of n_local workers' gradients (Algorithm 3: RHT, truncation,
 * stochastic quantisation, table index; Section 3: packing).  Worker i of this call is
 * worker (worker_base + i) of the job: its id keys its random stream, so that workers
 * round independently (Appendix A.2) while sharing D.
 *   scales   device, from thc_prepare (or any agreed positive bounds)
 *   packed   host array of n_local device pointers, packed_bytes each, written
 *   rotated  NULL, or host array of n_local device pointers (NULL entries allowed), each
 *            rotated_bytes: receives RHT(x_i), e.g. for error feedback or for tests      */
int thc_compress(thc_ctx *ctx, const void *const *grads, uint32_t n_local, uint32_t worker_base,
                 uint64_t d, uint32_t round, const float *scales, void *const *packed,
                 float *const *rotated, void *workspace, uint64_t workspace_bytes,
                 void *stream);

/* The quantisation half of thc_compress alone (Algorithm 2, worker lines 1-4, after the
 * truncation of Algorithm 3), on coordinates that are already rotated:
 *   rotated  host array of n_local device pointers, d_pad fp32 each, read                */
int thc_quantize_rotated(thc_ctx *ctx, const float *const *rotated, uint32_t n_local,
                         uint32_t worker_base, uint64_t d, uint32_t round, const float *scales,
                         void *const *packed, void *stream);

/* Parameter-server aggregation (Algorithm 2, PS line: Y = sum_i T[Z_i]; Section 3: lookups
 * and integer sums only).  n may be smaller than cfg.workers (partial aggregation, Section 6).
 *   packed  host array of n device pointers, read
 *   sum     device, sum_bytes, written                                                   */
int thc_aggregate(thc_ctx *ctx, const void *const *packed, uint32_t n, uint64_t d,
                  void *sum, void *stream);

/* Worker-side decompression (Algorithm 2: Y_avg = Y / n, estimate = m + Y_avg (M - m)/g;
 * Algorithm 3: inverse RHT).  `divisor` is the number of workers that were summed.
 *   out  device, d fp32, written                                                         */
int thc_decompress(thc_ctx *ctx, const void *sum, uint32_t divisor, uint64_t d, uint32_t round,
                   const float *scales, float *out, void *workspace, uint64_t workspace_bytes,
                   void *stream);

/* thc_aggregate followed by thc_decompress as one call, for a caller that holds all n workers'
 * packed indices on this GPU (the simulated cluster): Algorithm 2's PS line, Y = sum_i T[Z_i],
 * feeding the worker's estimate line and the inverse RHT (Algorithm 3) directly.  For RHT blocks
 * above 2^14 coordinates, 4-bit indices and table values below 128 this is one launch and the
 * sums never travel through memory; they are written (d_pad unsigned integers of acc_bits bits,
 * as thc_aggregate writes them) only if sum_or_null is given.  Elsewhere the call runs
 * thc_aggregate and thc_decompress (sums in the workspace unless a buffer is given).  `out` is bit for bit what the two calls give with divisor n.  The paper's
 * PS is another machine, so the separate calls remain the general form.
 *   packed       host array of n device pointers (n <= thc_config.workers)
 *   out          device, d fp32, written
 *   sum_or_null  device, sum_bytes, written if not NULL                                      */
int thc_aggregate_decompress(thc_ctx *ctx, const void *const *packed, uint32_t n, uint64_t d,
                             uint32_t round, const float *scales, float *out, void *sum_or_null,
                             void *workspace, uint64_t workspace_bytes, void *stream);

/* Preliminary stage without any allocation, for callers that may not call cudaMalloc (a
 * plugin inside a host framework's fixed memory plan, code running under a frozen memory
 * budget) and so can use neither thc_create (which allocates the context's device block)
 * nor a workspace of their own.  The paper has no counterpart of this entry point: it is
 * thc_prepare with the parameters passed as plain arguments and the fp64 partial sums kept
 * in a fixed array inside the library's device image (THC_NOALLOC_SCRATCH_BYTES on every
 * GPU that loads the library, until the process exits).
 *   grads            host array of n device pointers (16-byte aligned), d elements each
 *   log2_block, in_dtype, t_p   as in thc_config
 *   scales           device, ceil(d / 2^log2_block) fp32, written; the values of thc_prepare up to
 *                    the last bit (the fp64 partial sums are added in another fixed order)
 *   status_or_null   device word that THC_STATUS_NONFINITE / THC_STATUS_ZERO_BLOCK are OR-ed
 *                    into, or NULL
 * Limit: n * ceil(d_pad / 2^min(log2_block,14)) partial sums must fit the array (524,288
 * of them), else THC_EWORKSPACE is returned and nothing is launched.  Calls cudaMalloc,
 * cudaFree or any allocating routine never.  The first call on a device looks up the
 * array's device address (cudaGetSymbolAddress); make that call before any stream capture.
 * All calls share the array: calls that overlap on the GPU race; calls on one stream do
 * not.  Nothing in the array has to be cleared between calls.  d > 2^40 is THC_EINVAL like
 * everywhere else; device ordinals of 64 and above are not served (THC_ECUDA). */
#define THC_NOALLOC_SCRATCH_BYTES (4u << 20)
int thc_prepare_noalloc(const void *const *grads, uint32_t n, uint64_t d, uint32_t log2_block,
                        uint32_t in_dtype, double t_p, float *scales, uint32_t *status_or_null,
                        void *stream);

/* The preliminary stage of Algorithm 1 ("m = min_i m_i, M = max_i M_i") applied per RHT block to
 * the rotated coordinates: scales[k] = min and scales[nblocks + k] = max over all n workers and
 * all coordinates of block k of RHT(x_i) for this `round` (the rotation depends on it).
 * Contexts in THC_RANGE_MINMAX mode only (THC_EUNSUPPORTED otherwise; thc_prepare is their
 * counterpart in THC_RANGE_NORM mode).  thc_compress, thc_quantize_rotated, thc_decompress and
 * thc_error_feedback of such a context read `scales` in this layout and use the range
 * [m, M] of Algorithm 2 as given: no coordinate is clamped.  Costs one transform pass over the
 * inputs.  A block with a non-finite rotated coordinate gets (0, 0) and THC_STATUS_NONFINITE.
 * rotated_or_null: host array of n device pointers (d_pad fp32 each) that receive the rotated
 * coordinates, so that thc_quantize_rotated can finish the compression without a second
 * transform; null (or a null entry) to skip. */
int thc_prepare_minmax(thc_ctx *ctx, const void *const *grads, uint32_t n, uint64_t d, uint32_t round,
                       float *scales, float *const *rotated_or_null, void *workspace,
                       uint64_t workspace_bytes, void *stream);

/* thc_prepare and thc_compress in one launch, for callers that hold all n workers' gradients
 * (the simulated cluster): same arguments and results as the two calls in a row, `scales`
 * (device, nblocks floats) being written here and usable by thc_decompress afterwards.
 * Section 5.3 observes that the norm exchange can overlap the RHT: only the quantiser needs M,
 * so where the block size is 2^20, the input fp32 and n small enough for the intermediate ring
 * to stay in L2, the transform kernel sums the squares of the tiles it loads anyway and the
 * gradients are read from HBM once instead of twice.  Elsewhere this runs the two calls.
 * The fp64 sums are added in a different (fixed) order than thc_prepare's, so a scale may
 * differ from thc_prepare's in the last bit.  */
int thc_prepare_compress(thc_ctx *ctx, const void *const *grads, uint32_t n, uint32_t worker_base,
                         uint64_t d, uint32_t round, float *scales, void *const *packed,
                         float *const *rotated_or_null, void *workspace, uint64_t workspace_bytes,
                         void *stream);

/* Error feedback (Section 5.1; Algorithm 3, "e_i = x_i - RHT^-1(X_i)"): for each of the n_local
 * workers, the residual between what it compressed and what its own indices stand for,
 *     ef[i] = x_i - RHT^-1( m + T[Z_i] (M - m)/g ),
 * to be added to the next round's gradient (thc_accumulate_error).  fp32 contexts only
 * (THC_EUNSUPPORTED for bf16 inputs).  For RHT blocks above 2^14 coordinates this is one launch
 * over all workers (indices in, de-quantised in registers, inverse transform, x - result out);
 * for smaller blocks it is composed per worker of thc_aggregate with n = 1, thc_decompress with
 * divisor 1 and one subtraction.  Both give the same bits.
 *   grads    host array of n_local device pointers: the x_i that were compressed
 *   packed   host array of n_local device pointers: their packed indices
 *   ef       host array of n_local device pointers, d fp32 each, written
 *   workspace  as reported by thc_sizes (it includes room for one worker's table values)  */
int thc_error_feedback(thc_ctx *ctx, const void *const *grads, const void *const *packed,
                       uint32_t n_local, uint64_t d, uint32_t round, const float *scales,
                       float *const *ef, void *workspace, uint64_t workspace_bytes, void *stream);

/* Algorithm 3, "x_i = grad_i + e_i": grads[i] += ef[i] in place, fp32, d elements each. */
int thc_accumulate_error(thc_ctx *ctx, float *const *grads, const float *const *ef,
                         uint32_t n_local, uint64_t d, void *stream);

/* Read and clear the status bits (synchronises `stream`).  flags is a host pointer. */
int thc_status(thc_ctx *ctx, uint32_t *flags, void *stream);

/* Test hook for the bounded waits of the large-block pipeline (no counterpart in the paper).
 * The next thc_compress / thc_decompress on this context starts its task queue at position
 * `count` instead of 0, so tasks that depend on the skipped ones can never be satisfied: the
 * kernel must notice (about one second), set THC_STATUS_WAIT_TIMEOUT, and return with the
 * context still usable; the outputs of that call are undefined.  Synchronises the device. */
int thc_debug_skip_tasks(thc_ctx *ctx, uint32_t count);

const char *thc_strerror(int code);

/* Library build identification, e.g. "thc-b200 sm_100a". */
const char *thc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* THC_H_ */
