/*
 * sradamw.h -- C ABI of libsradamw.so: the BF16 + stochastic-rounding AdamW update on one B200.
 *
 * The update is Algorithm 1 ("AdamW with Stochastic Rounding and Shared Randomness"): parameters x,
 * gradients g and both moments m, v are stored in BF16; one iteration reads them, evaluates the
 * AdamW formulas in FP32 registers and writes x, m, v back to BF16 with stochastic rounding Q_SR
 * (Eq. 2), implemented the way Section 3 describes: add uniform noise below the kept bits of the
 * FP32 pattern, then drop the low half.  No FP32 master copy and no auxiliary tensor exists.
 *
 * Conventions for every call
 *   - Data pointers are DEVICE pointers owned by the caller unless a parameter says "host".
 *     BF16 arrays are passed as uint16_t bit patterns.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls enqueue work and
 *     return; they never synchronise the device and never allocate device memory, except
 *     sr_mt_plan_create / sr_mt_plan_destroy.
 *   - The step kernels keep their staging in more shared memory than a kernel gets by default: the first call that
 *     needs a kernel variant on a device sets that kernel's attribute (cudaFuncSetAttribute; nothing is allocated).
 *     Make the first call of a configuration outside any stream capture.
 *   - x, m, v are updated in place; g is only read.  Buffers of one call must not overlap each other.
 *   - n == 0 is a successful no-op.  Any base alignment is accepted; the 16-byte vector path needs
 *     all buffers of a call 16-byte aligned and otherwise an element-wise path is taken.
 *   - Errors are returned, never thrown; nothing is written when a call returns an error other
 *     than SR_ERR_CUDA.  The device must have compute capability 10.x.
 *
 * The optimizer's random state (Algorithm 1: r^(opt)_t, equal on every replica) is a pure function
 * of the arguments.  With index = elem_offset + position in the buffer, one Philox4x32-10 call
 * serves one rounding slot (0: x, 1: m, 2: v) of a group of eight consecutive indices:
 *   number  = 4 * (index >> 3) + slot                         (64-bit)
 *   key     = (seed[31:0], step)
 *   counter = (number[31:0], number[63:32], tensor_id, seed[63:32])
 * Element e = index & 7 uses output word e >> 1, its low 16 bits if e is even, its high 16 bits if
 * e is odd; every bit of every call is used once.  sr_downcast_f32_bf16 uses slot 0,
 * sr_accumulate_bf16 slot 3; the FP8 / FP4 casts draw 32 bits per element (layout stated there).
 * Two ranks, two shards or two runs with equal (seed, step, tensor_id, index) therefore round
 * identically, which is what the shared random state of Algorithm 1 is for.
 */
#ifndef SRADAMW_H
#define SRADAMW_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SR_ABI_VERSION 1u

typedef enum {
    SR_OK = 0,
    SR_ERR_INVALID_ARG = 1,        /* null pointer, step 0 for AdamW, bad hyper-parameter or struct size */
    SR_ERR_UNSUPPORTED_DEVICE = 2, /* current device is not compute capability 10.x                      */
    SR_ERR_WORKSPACE = 3,          /* workspace missing or too small                                     */
    SR_ERR_CUDA = 4                /* a CUDA runtime call failed; see sr_last_cuda_error()                */
} sr_status;

typedef enum { SR_DT_BF16 = 0, SR_DT_F32 = 1 } sr_dtype; /* gradient storage; x, m, v are always BF16 */

/* flags of sr_adamw_hparams: which of the three downcasts use Q_SR (Eq. 2); the others use
 * round-to-nearest-even (Eq. 1).  Algorithm 1 itself needs SR_FLAG_SR_P only. */
#define SR_FLAG_SR_P 1u
#define SR_FLAG_SR_M 2u
#define SR_FLAG_SR_V 4u
#define SR_FLAGS_DEFAULT 7u
/* Where epsilon sits in the update step.  Algorithm 1 as printed takes a square root in its v-hat
 * step and divides by sqrt(v-hat + eps) in the update step, which read literally is a double root.
 * Default (flag clear): the AdamW of the optimizer the paper cites, den = sqrt(v/(1-beta2^t)) + eps.
 * SR_FLAG_EPS_INSIDE: the form the paper's analysis uses (appendix: m / sqrt(eps + v)), with the
 * bias correction kept: den = sqrt(v/(1-beta2^t) + eps), evaluated as sqrt(fma(v, 1/(1-beta2^t), eps)).
 * Both readings run the same branch-free kernels at the same speed. */
#define SR_FLAG_EPS_INSIDE 8u

/* Hyper-parameters of one iteration (Algorithm 1, REQUIRE list).  Host memory, read during the call. */
typedef struct sr_adamw_hparams {
    uint32_t struct_size;        /* sizeof(sr_adamw_hparams); checked                                        */
    float lr;                    /* alpha_t, finite, >= 0                                                     */
    float beta1;                 /* in [0, 1)                                                                 */
    float beta2;                 /* in [0, 1)                                                                 */
    float eps;                   /* finite, >= 0; added to sqrt(v-hat), outside the square root               */
    float weight_decay;          /* lambda, finite; decoupled: the decay term is alpha_t * lambda * x          */
    float grad_scale;            /* g is multiplied by this before use when grad_scale_dev is NULL (1 = none) */
    const float* grad_scale_dev; /* optional DEVICE scalar (e.g. from sr_clip_scale); read by the kernel       */
    uint32_t flags;              /* SR_FLAG_SR_* | SR_FLAG_EPS_INSIDE; other bits must be zero                 */
} sr_adamw_hparams;

/* Eq. 2 on an array: dst[i] = Q_SR(src[i]) using slot 0 of the noise at index elem_offset + i.
 * src: n FP32 values; dst: n BF16 patterns.  step may be 0 here.
 * NaN inputs give the quiet NaN 0x7FC0; +-0, +-inf and values already representable pass through. */
sr_status sr_downcast_f32_bf16(const float* src, uint16_t* dst, uint64_t n, uint64_t seed, uint32_t step,
                               uint32_t tensor_id, uint64_t elem_offset, void* stream);

/* Eq. 2 onto an 8-bit floating-point grid (the extension the paper's conclusion names): dst[i] =
 * Q_SR(src[i]) with the two neighbouring levels taken from E4M3 (bias 7, no infinity, largest finite
 * 448, NaN = S.1111.111) or E5M2 (bias 15, IEEE-like, largest finite 57344).  With a = |x| in the
 * binade Eq = max(E, 1 - bias), y = a / 2^(Eq - M) = k + f: the value moves to level k + 1 iff
 * r < floor(f * 2^32) for a uniform 32-bit r, i.e. with probability f (exact whenever f has at most
 * 32 fractional bits).  Magnitudes at or beyond the largest finite level saturate to it (E5M2 keeps
 * +-inf), NaN gives 0x7F.  Noise: one Philox call per four consecutive indices, counter number =
 * index >> 2 (other counter and key words as above), element index & 3 takes output word index & 3.
 * src: n FP32 values; dst: n bytes.  A call whose indices cross a multiple of 2^34 is enqueued as one
 * launch per stretch, in order on the stream (sr_downcast_f32_fp4 likewise). */
typedef enum { SR_FP8_E4M3 = 0, SR_FP8_E5M2 = 1 } sr_fp8_format;
sr_status sr_downcast_f32_fp8(const float* src, uint8_t* dst, uint64_t n, sr_fp8_format format, uint64_t seed,
                              uint32_t step, uint32_t tensor_id, uint64_t elem_offset, void* stream);

/* Eq. 2 onto the 4-bit floating-point grid E2M1 (the conclusion names FP8 and FP4): one sign bit, 2
 * exponent bits with bias 1, one mantissa bit; magnitudes 0, 0.5, 1, 1.5, 2, 3, 4, 6 are codes 0..7,
 * bit 3 is the sign.  Same rule and same noise as sr_downcast_f32_fp8 with M = 1, bias = 1.  The
 * format has neither infinity nor NaN: every magnitude at or beyond 6 gives +-6, infinity included,
 * and a NaN gives the largest magnitude with its sign bit (a choice of this library; the paper is
 * silent).  src: n FP32 values; dst: (n + 1) / 2 bytes, element 2j in bits 0..3 and element 2j + 1
 * in bits 4..7 of byte j (the upper half of the last byte is 0 when n is odd). */
sr_status sr_downcast_f32_fp4(const float* src, uint8_t* dst, uint64_t n, uint64_t seed, uint32_t step,
                              uint32_t tensor_id, uint64_t elem_offset, void* stream);

/* Eq. 2 (or Eq. 1) in a BF16 accumulation, e.g. of micro-batch gradients (Section 3: every tensor
 * is BF16): acc[i] <- rounding(acc[i] + scale * g[i]) with the product and the sum each one FP32
 * operation.  flags = SR_FLAG_SR_P rounds stochastically, flags = 0 to nearest-even; other bits are
 * rejected.  Noise: rounding slot 3 of the layout above (counter number 4 * (index >> 3) + 3), which
 * sr_adamw_step never draws, so the same (seed, step, tensor_id) may be shared with the step; the
 * caller gives every accumulation of one iteration its own `step` value (or seed).  step may be 0.
 * acc: n BF16 in/out; g: n BF16 or FP32 values per g_dtype, read-only; scale: finite. */
sr_status sr_accumulate_bf16(uint16_t* acc, const void* g, sr_dtype g_dtype, uint64_t n, float scale, uint32_t flags,
                             uint64_t seed, uint32_t step, uint32_t tensor_id, uint64_t elem_offset, void* stream);

/* One iteration of Algorithm 1 on a flat buffer of n elements (moment updates, bias-corrected
 * direction with epsilon outside the square root, decoupled weight decay, rounding of x, m, v).
 * p, m, v: BF16 in/out.  g: BF16 or FP32 per g_dtype.  step >= 1 is the 1-based iteration t.
 * elem_offset is the global index of element 0, so a shard of a larger buffer rounds as the whole
 * buffer would.  Fastest when all four buffers are 16-byte aligned and elem_offset is a multiple of
 * 8 (shards cut at multiples of 8 elements); other offsets and alignments give the same bits through
 * slower kernels (an offset that is not a multiple of 8 doubles the Philox calls and costs about a
 * quarter of the throughput). */
sr_status sr_adamw_step(uint16_t* p, const void* g, sr_dtype g_dtype, uint16_t* m, uint16_t* v, uint64_t n,
                        const sr_adamw_hparams* hp, uint64_t seed, uint32_t step, uint32_t tensor_id,
                        uint64_t elem_offset, void* stream);
/* Number of kernel launches one sr_adamw_step call of n elements at elem_offset enqueues: the call is cut into
 * launches of 2^28 elements (the last one up to 1.5 times that), none crossing a multiple of 2^33 in index
 * space.  The cuts change nothing in the result.  Host-only. */
uint32_t sr_adamw_step_launch_count(uint64_t n, uint64_t elem_offset);

/* The mixed-precision recipe the paper compares against (Section 3: FP32 master weights and FP32
 * optimizer states, BF16 copy of the weights), provided so that both recipes can be measured with
 * the same arithmetic on the same GPU.  p, m, v: FP32 in/out; p_bf16: BF16 copy of the updated x,
 * rounded to nearest (Eq. 1), written only; g: BF16 or FP32.  Same element function as
 * sr_adamw_step, no noise; hp->flags is ignored.  28 (30) bytes per element instead of 14 (16). */
sr_status sr_master_adamw_step(float* p, uint16_t* p_bf16, const void* g, sr_dtype g_dtype, float* m, float* v,
                               uint64_t n, const sr_adamw_hparams* hp, uint32_t step, void* stream);

/* The same iteration for state that lives in HOST memory (optimizer state kept off the device):
 * the buffer is cut into chunks; each chunk is copied host->device into `staging`, stepped by the
 * same kernel as sr_adamw_step (with elem_offset advanced, so the result equals the in-device
 * step bit for bit) and its x, m, v copied back.  Two chunks are in flight on two streams (the
 * caller's and one the library keeps per device) so uploads, kernels and downloads overlap.
 * p, g, m, v: HOST pointers, page-locked for the copies to be asynchronous; they must stay valid
 * until `stream` has been synchronised.  staging: DEVICE scratch, 256-byte aligned, at least
 * sr_adamw_step_host_staging_bytes(g_dtype, chunk_elems) bytes, chunk_elems a non-zero multiple of
 * 8; larger chunks amortise copy latency (2^24 elements is a reasonable choice).
 * grad_scale_dev, if set, stays a device pointer.  The first call on a device creates the
 * library's second stream and two events (kept until the process ends); calls from several host
 * threads are serialised while they enqueue. */
size_t sr_adamw_step_host_staging_bytes(sr_dtype g_dtype, uint64_t chunk_elems);
sr_status sr_adamw_step_host(uint16_t* p_host, const void* g_host, sr_dtype g_dtype, uint16_t* m_host,
                             uint16_t* v_host, uint64_t n, const sr_adamw_hparams* hp, uint64_t seed, uint32_t step,
                             uint32_t tensor_id, uint64_t elem_offset, void* staging, size_t staging_bytes,
                             uint64_t chunk_elems, void* stream);

/* The same iteration over a list of tensors: one launch for all tensors below 2^24 elements (and for those
 * whose buffers are not 16-byte aligned), plus one launch of the flat kernel per larger tensor, all enqueued by
 * the one call and all ordered inside `stream`: they start after the work enqueued on `stream` before the call
 * and whatever is enqueued on it afterwards starts after them.  With two or more large tensors every second
 * flat launch runs on a stream that the plan owns, forked from and joined to `stream` by events inside the call (the
 * tensors are disjoint, so the end of one launch overlaps the start of the next; the pattern can be captured in a
 * CUDA graph).  One host thread at a time may step a given plan.  A plan owns a device copy of the chunk table
 * that maps thread blocks to (tensor, range), the host-side list of the large tensors, and that stream.
 * The arrays passed to sr_mt_plan_create are HOST arrays of num_tensors entries holding device
 * pointers and element counts; they may be freed after the call.  Tensor i uses
 * tensor_id = tensor_id_base + i and element indices starting at 0.  One hparams set serves the list.
 * The plan stays valid while the tensors it names stay allocated; destroy it with
 * sr_mt_plan_destroy (which synchronises nothing: do not destroy while a step using it is in flight).
 * A plan belongs to the device that was current when it was created: sr_adamw_multi_tensor returns
 * SR_ERR_INVALID_ARG under another current device.  Creation returns SR_ERR_WORKSPACE when host or
 * device memory for the tables cannot be had. */
typedef struct sr_mt_plan sr_mt_plan;
sr_status sr_mt_plan_create(sr_mt_plan** out, uint32_t num_tensors, uint16_t* const* p, const void* const* g,
                            uint16_t* const* m, uint16_t* const* v, const uint64_t* numel, sr_dtype g_dtype,
                            void* stream);
sr_status sr_adamw_multi_tensor(const sr_mt_plan* plan, const sr_adamw_hparams* hp, uint64_t seed, uint32_t step,
                                uint32_t tensor_id_base, void* stream);
sr_status sr_mt_plan_destroy(sr_mt_plan* plan);
uint64_t sr_mt_plan_total_elements(const sr_mt_plan* plan);

/* Sum of squares of the gradient for global-norm clipping (not part of the paper; the usual
 * companion of the update).  The sum is taken in FP64 over exact squares with a fixed tree that
 * does not depend on the launch shape: blocks of 8192 consecutive entries; inside a block 256
 * accumulators, accumulator j adding entries r*1024 + 4j + k (r = 0..7, k = 0..3) in that order;
 * 8 groups of 32 accumulators folded by an XOR butterfly (16, 8, 4, 2, 1), group values added in
 * order; the block sums are reduced again by the same rule until one value is left.
 * out_dev: one double on the device; while the call's kernels run it holds a count of finished blocks
 * (n > 2^26), so nothing else may read it before they have completed.  workspace: device memory of at
 * least grad_sqnorm_workspace_bytes(n) bytes, 8-byte aligned (may be NULL when that size is 0). */
size_t grad_sqnorm_workspace_bytes(uint64_t n);
sr_status grad_sqnorm(const void* g, sr_dtype g_dtype, uint64_t n, double* out_dev, void* workspace,
                      size_t workspace_bytes, void* stream);

/* The same sum over the gradients of a tensor list (global-norm clipping of a whole model; not part
 * of the paper either).  The first pass takes one block sum per chunk of the plan: tensor by tensor
 * in list order, every tensor cut into chunks of 8192 consecutive entries (the last one ragged), the
 * block rule above applied inside each chunk with positions counted from the chunk's start.  The
 * array of block sums, in that order, is then reduced by the later passes of grad_sqnorm.  For a
 * list of one tensor the result equals grad_sqnorm's, bit for bit; so it does for a list whose
 * tensors all have lengths that are multiples of 8192, against grad_sqnorm of their concatenation.
 * out_dev: one double on the device (as in grad_sqnorm it is the call's own counter while its kernels run,
 * for lists of more than 8192 chunks).  workspace: device memory of at least
 * grad_sqnorm_multi_tensor_workspace_bytes(plan) bytes, 8-byte aligned (may be NULL when that is 0).
 * Reads the gradient pointers the plan was created with; call under the plan's device. */
size_t grad_sqnorm_multi_tensor_workspace_bytes(const sr_mt_plan* plan);
sr_status grad_sqnorm_multi_tensor(const sr_mt_plan* plan, double* out_dev, void* workspace, size_t workspace_bytes,
                                   void* stream);

/* grad_sqnorm for callers that cannot allocate.  (The paper has no counterpart; neither has the
 * rest of the norm/clipping code.)  Some users of this library run where cudaMalloc is not an
 * option: inside a process whose device memory is owned and fully handed out by someone else's
 * pool, inside a callback or a latency-critical loop where an allocation (or the synchronisation it
 * can imply) is forbidden, or in a harness that is only allowed to pass its inputs and outputs.
 * For them the intermediate block sums live in a fixed 1 MiB array (131 072 doubles) inside the
 * library image; every GPU that loads the library holds that array until the process exits.
 *   - Same result as grad_sqnorm, bit for bit (same kernels, same tree).
 *   - n may be at most grad_sqnorm_static_max_elements() (1 073 610 752: enough for a 1/8 shard of
 *     the 6.7B model); larger n returns SR_ERR_WORKSPACE and nothing is launched.
 *   - The call allocates nothing and frees nothing.  Its FIRST call on each device looks up the
 *     array's device address (a one-off set-up); make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps what the previous call left in it.
 *     Nothing in it has to be zero beforehand, because every block sum is written before it is
 *     read within a call.  Two calls that can overlap on the GPU (different streams, no ordering
 *     between them) would overwrite each other's block sums: order them, or give one of them its
 *     own workspace through grad_sqnorm. */
uint64_t grad_sqnorm_static_max_elements(void);
sr_status grad_sqnorm_static(const void* g, sr_dtype g_dtype, uint64_t n, double* out_dev, void* stream);

/* Clipping factor on the device, no host round trip:
 * gscale = accum_scale * min(1, max_norm / (accum_scale * sqrt(S) + 1e-6)), evaluated in FP64 and
 * stored as FP32 in *gscale_out_dev; pass that pointer as sr_adamw_hparams.grad_scale_dev. */
sr_status sr_clip_scale(const double* sqnorm_dev, float accum_scale, float max_norm, float* gscale_out_dev,
                        void* stream);

/* Self-check of the step kernels' arithmetic.  Algorithm 1's update divides the first moment by the root of the
 * second (its last two lines); the fused kernels evaluate that square root and that division with fixed
 * sequences of FP32 multiply-adds on the hardware's reciprocal / reciprocal-root seeds, which equal the IEEE
 * round-to-nearest results inside the operand range the kernels check per vector (argument of the root and
 * |numerator| in [2^-60, 2^60], denominator in [2^-30, 2^41]).  This call draws `sets` operand sets from
 * Philox4x32-10 keyed by `seed` -- exponents uniform over those ranges; mantissas plain, just below a power of
 * two or just above one; and denominators formed the way the kernels form them -- evaluates both forms and
 * counts the results that differ: mismatches_dev[0] square roots, mismatches_dev[1] divisions (device memory,
 * two uint64_t, overwritten).  Both counts are expected to be 0; the square root has also been compared on
 * every FP32 value of its range. */
sr_status sr_selftest_in_range_arithmetic(uint64_t seed, uint64_t sets, uint64_t* mismatches_dev, void* stream);

const char* sr_status_string(sr_status s);
int sr_last_cuda_error(void); /* cudaError_t of the last failing runtime call on this thread, else 0 */
uint32_t sr_abi_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SRADAMW_H */
