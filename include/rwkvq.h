/*
 * rwkvq -- hybrid scalar/vector-quantized RWKV projection products on NVIDIA B200 (sm_100a).
 *
 * C ABI of the library.  Every entry point returns a status code; nothing aborts,
 * throws or traps.  Pointers named *_host are host memory, pointers named *_dev
 * are device memory owned by the caller (the library never allocates device
 * memory in any call declared here unless the comment says so).  `stream` is a
 * cudaStream_t passed as void* (NULL = the legacy default stream).  Kernels are
 * asynchronous on `stream`; argument errors are detected on the host before any
 * launch.
 *
 * Method references are to RWKVQuant (arXiv 2505.03803): scalar quantization
 * Section 3.2 Eq. 2, vector quantization Section 3.2 Eq. 3, coarse-to-fine proxy
 * Section 4.1 Eqs. 5-18, element-wise (token-shift) weights Section 4.2 and
 * Appendix A.1 Eqs. 20-27.
 */
#ifndef RWKVQ_H_
#define RWKVQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RWKVQ_OK = 0,
  RWKVQ_EINVAL = 1,       /* NULL pointer, bad enum, bad size */
  RWKVQ_ESHAPE = 2,       /* shape not supported by the format (see rwkvq_pack) */
  RWKVQ_EALIGN = 3,       /* a device pointer is not 16-byte aligned */
  RWKVQ_ENONFINITE = 4,   /* NaN/Inf in the weights */
  RWKVQ_ENOMEM = 5,       /* host allocation failed, or caller buffer / workspace too small */
  RWKVQ_ECUDA = 6,        /* a CUDA runtime call failed (see rwkvq_last_cuda_error) */
  RWKVQ_EUNSUPPORTED = 7, /* valid request this build does not implement */
  RWKVQ_ETIMEOUT = 8      /* a bounded device-side wait expired (reported by rwkvq_device_status) */
} rwkvq_status;

/* phi_m of Section 4.1 Eq. 18: 1 = scalar quantization, 0 = vector quantization. */
typedef enum { RWKVQ_VQ = 0, RWKVQ_SQ = 1 } rwkvq_method;

typedef enum { RWKVQ_F32 = 0, RWKVQ_F16 = 1, RWKVQ_BF16 = 2 } rwkvq_dtype;

/*
 * Logical (format-independent) codes of one matrix, host memory.
 *  SQ (Eq. 2):  q[oc*ic] codes in [0, 2^bits-1] row-major; scale/zero: fp16 bit
 *               patterns, [oc * ic/group], one pair per run of `group` consecutive
 *               input-dim weights of one row.  Decode: w_hat = s * (q - z).
 *  VQ (Eq. 3):  q[oc*ic/2] codebook indices row-major (vector = two consecutive
 *               input-dim weights of one row); codebook: fp16 bit patterns
 *               [oc/tile][ic/tile][2^bits][2], one codebook per tile x tile block.
 *               Decode: w_hat[i][2p+e] = C_tile(i,p)[q[i][p]][e].
 *  mu vectors (oc == 1, VQ): one codebook [2^bits][2], q[ic/2].
 * Unused members are NULL.
 */
typedef struct {
  uint8_t* q;
  uint16_t* scale;
  uint16_t* zero;
  uint16_t* codebook;
} rwkvq_codes;

typedef struct {
  int32_t method;       /* rwkvq_method */
  int32_t bits;         /* SQ: code bits, 3.  VQ: index bits, 6 (64 entries) or 8 (256 entries) */
  int32_t group;        /* SQ: 128 */
  int32_t vec_dim;      /* VQ: 2 */
  int32_t tile;         /* VQ: 256 (ignored for oc == 1) */
  int32_t kmeans_iters; /* VQ: Lloyd iterations after k-means++ seeding, e.g. 10 */
  uint64_t seed;        /* VQ: seed of the library's own generator */
  const rwkvq_codes* codes_in; /* optional: pre-made logical codes; the quantizer is skipped
                                  and the codes are packed as given (w_fp16_host may be NULL) */
} rwkvq_quant_cfg;

/* Host-side description of a packed matrix; travels with the device image. */
typedef struct {
  int32_t method, bits, oc, ic, group, vec_dim, tile, entries;
  int32_t oc_pad, ic_pad;  /* rows padded to 128, columns to 256 inside the image */
  uint64_t image_bytes;    /* size of the device image, multiple of 256 */
  uint64_t stream_bytes;   /* bytes a product must read: codes + scales / indices + codebooks */
} rwkvq_desc;

typedef struct rwkvq_blob rwkvq_blob; /* host-owned packed matrix, opaque */

/*
 * Quantize (unless cfg->codes_in) and bit-pack one fp16 matrix W[oc][ic] (row-major, rows =
 * output channels, host memory, fp16 bit patterns).  SQ follows Eq. 2 with s = (max-min)/(2^b-1)
 * rounded to fp16, integer zero point z = round(-min/s) and round-to-nearest-even; VQ follows
 * Eq. 3 with a k-means codebook per tile (Section 3.2).  Token-shift vectors (Section 4.2) are
 * packed with oc = 1, method = RWKVQ_VQ.
 * Shapes: SQ needs oc % 16 == 0 and ic % 128 == 0; VQ matrices need oc % 256 == 0 and
 * ic % 256 == 0; vectors need ic % 2 == 0.  Errors: EINVAL, ESHAPE, ENONFINITE, ENOMEM.
 * On success *out owns host memory until rwkvq_blob_free.
 */
rwkvq_status rwkvq_pack(const uint16_t* w_fp16_host, int oc, int ic, const rwkvq_quant_cfg* cfg,
                        rwkvq_blob** out);
rwkvq_status rwkvq_blob_desc(const rwkvq_blob* blob, rwkvq_desc* desc_out);
/* Size of the device image in bytes (multiple of 256; 0 for NULL). */
size_t rwkvq_blob_nbytes(const rwkvq_blob* blob);
/* Copy the device image (header + bit-packed payload) into dst_host[n]; the caller then copies
 * it to a 256-byte-aligned device buffer.  ENOMEM if n is too small. */
rwkvq_status rwkvq_blob_image(const rwkvq_blob* blob, void* dst_host, size_t n);
/* Copy the logical codes into caller-allocated arrays (sizes as in rwkvq_codes). */
rwkvq_status rwkvq_blob_export_codes(const rwkvq_blob* blob, rwkvq_codes* dst_host);
/* Unpack a host copy of a device image back into logical codes (inverse of the bit packing;
 * checks magic, version, sizes and CRC).  desc_out may be NULL; dst arrays as in rwkvq_codes. */
rwkvq_status rwkvq_image_unpack(const void* image_host, size_t n, rwkvq_desc* desc_out,
                                rwkvq_codes* dst_host);
void rwkvq_blob_free(rwkvq_blob* blob);

/*
 * Coarse-to-fine proxy (Section 4.1).  For each of n_mats fp16 matrices resident on the device
 * computes P_c (Eq. 9) and P_f (Eq. 17, orders 2..K, 2 <= K <= 8) from the sorted-gap
 * distribution of the flattened weights and applies Eq. 18:
 * phi = 1 (SQ) iff P_c < tau_c and P_f < tau_f, else 0 (VQ).  A constant matrix yields
 * P_c = P_f = +inf (VQ).  Pc_host/Pf_host/phi_host: host arrays of n_mats (written after the
 * call synchronizes `stream`).  workspace_dev: at least rwkvq_proxy_workspace_bytes(n_mats) bytes,
 * 16-byte aligned; its contents on entry are irrelevant.  Errors: EINVAL, EALIGN, ENOMEM,
 * ENONFINITE (a NaN/Inf weight was seen), ECUDA.
 */
size_t rwkvq_proxy_workspace_bytes(int n_mats);
rwkvq_status rwkvq_proxy_select(const void* const* w_fp16_dev, const int* oc, const int* ic,
                                int n_mats, int K, double tau_c, double tau_f, double* Pc_host,
                                double* Pf_host, int* phi_host, void* workspace_dev,
                                size_t workspace_bytes, void* stream);

/*
 * The same proxy for weights of other types and at finer granularity (Section 4.1 evaluates one
 * matrix at a time; the paper's limitations paragraph names finer granularity as future work).
 *
 * rwkvq_proxy_select_bf16: as rwkvq_proxy_select for bfloat16 matrices (the sort of Eq. 5 as a
 * counting sort over the 65 536 bfloat16 patterns); same workspace size and errors.
 *
 * rwkvq_proxy_select_f32: one fp32 matrix resident on the device; the sort of Eq. 5 is the CUDA
 * toolkit's radix sort, the gaps are reduced in fp64 in a fixed order.  workspace_dev:
 * rwkvq_proxy_f32_workspace_bytes(oc, ic) bytes (two key arrays and the sort's scratch),
 * 256-byte aligned.  Pc_host/Pf_host/phi_host: one value each.
 *
 * rwkvq_proxy_segments: P_c, P_f and Eq. 18 for every seg_rows x seg_cols tile of one matrix
 * (dtype RWKVQ_F16, RWKVQ_BF16 or RWKVQ_F32, row-major [oc][ic] on the device): seg_rows = 1,
 * seg_cols = ic is channel level, 256 x 256 the block of a VQ codebook; tiles at the right and
 * bottom edges are smaller.  A tile is sorted by one thread block in shared memory, so it may hold
 * at most 65 536 elements (16-bit types) or 32 768 (fp32): EUNSUPPORTED beyond.  Results are
 * written tile-row major: index (r / seg_rows) * ceil(ic / seg_cols) + c / seg_cols; a tile with
 * fewer than two elements, or constant, yields +inf (VQ).  workspace_dev:
 * rwkvq_proxy_segments_workspace_bytes() bytes, 16-byte aligned.
 * All three synchronize `stream` before returning.  Errors: EINVAL, EALIGN, ENOMEM,
 * EUNSUPPORTED, ENONFINITE (the affected results are +inf), ECUDA.
 */
rwkvq_status rwkvq_proxy_select_bf16(const void* const* w_bf16_dev, const int* oc, const int* ic,
                                     int n_mats, int K, double tau_c, double tau_f, double* Pc_host,
                                     double* Pf_host, int* phi_host, void* workspace_dev,
                                     size_t workspace_bytes, void* stream);
size_t rwkvq_proxy_f32_workspace_bytes(int oc, int ic);
rwkvq_status rwkvq_proxy_select_f32(const void* w_f32_dev, int oc, int ic, int K, double tau_c,
                                    double tau_f, double* Pc_host, double* Pf_host, int* phi_host,
                                    void* workspace_dev, size_t workspace_bytes, void* stream);
size_t rwkvq_proxy_segments_workspace_bytes(int oc, int ic, int seg_rows, int seg_cols);
rwkvq_status rwkvq_proxy_segments(const void* w_dev, int dtype, int oc, int ic, int seg_rows,
                                  int seg_cols, int K, double tau_c, double tau_f, double* Pc_host,
                                  double* Pf_host, int* phi_host, void* workspace_dev,
                                  size_t workspace_bytes, void* stream);

/*
 * The statistics of the normalised gaps G' (Eq. 6) that the ablation of Section 5.3 tries in the
 * proxy's place, from the same histogram pass: for each matrix stats_host[5*m + {0,1,2,3,4}] =
 * variance, coefficient of variation, range, mean absolute deviation of G' and its information
 * entropy -sum G' ln G' (P_c = ln n - entropy).  A constant matrix yields +inf for all five.
 * Arguments and errors as rwkvq_proxy_select (same workspace size).
 */
rwkvq_status rwkvq_proxy_family(const void* const* w_fp16_dev, const int* oc, const int* ic, int n_mats,
                                double* stats_host, void* workspace_dev, size_t workspace_bytes,
                                void* stream);
/*
 * Threshold that sends the share sq_fraction of n matrices to scalar quantization under the rule
 * "SQ iff value < tau" (Section 5.1 sets the thresholds so that nine tenths of the layers use SQ):
 * with the values sorted and k = round(sq_fraction * n), tau is halfway between the k-th and the
 * (k+1)-th smallest; k = 0 gives -inf, k = n gives +inf.  Host only.  Errors: EINVAL (NULL,
 * n <= 0, fraction outside [0, 1], NaN among the values).
 */
rwkvq_status rwkvq_tau_for_fraction(const double* values_host, int n, double sq_fraction, double* tau_out);
/*
 * Threshold for the same rule when the values fall into two clusters (the synthetic stacks mix
 * Gaussian and heavy-tailed matrices, whose coarse proxies P_c of Eq. 9 are far apart): the
 * midpoint of the widest gap between neighbouring finite values in sorted order, the first such
 * gap when several are equally wide.  Fewer than two finite values, or all of them equal, give
 * +inf (everything scalar-quantized).  Host only.  Errors: EINVAL (NULL, n <= 0, NaN among the values).
 */
rwkvq_status rwkvq_tau_largest_gap(const double* values_host, int n, double* tau_out);

/*
 * Decode product y[b][i] = sum_j w_hat[i][j] * x_mix[b][j], 1 <= B <= 16 (Appendix A.1, the
 * W.(...) products), with the token-shift mix x_mix = x + (x_prev - x) (.) mu_hat fused into the
 * input stage when mu_image_dev != NULL (Eq. 20 with mu_paper = 1 - mu_hat).
 *  W_desc/W_image_dev: packed matrix and its description.  mu_desc/mu_image_dev: packed vector of
 *  length ic, or both NULL.  x_fp16_dev, xprev_fp16_dev: [B][ic] fp16 (xprev NULL iff mu NULL).
 *  y_dev: [B][oc], y_dtype F32 or F16.  workspace_dev: rwkvq_gemv_workspace_bytes() bytes, must
 *  be zero-filled once before its first use; later calls may reuse it without clearing (each call
 *  restores the part that has to be zero), but calls that share a workspace must not overlap on
 *  the device.
 * Accumulation is fp32.  Errors: EINVAL, ESHAPE, EALIGN, ENOMEM, ECUDA.
 */
size_t rwkvq_gemv_workspace_bytes(const rwkvq_desc* W_desc, int B);
rwkvq_status rwkvq_gemv(const rwkvq_desc* W_desc, const void* W_image_dev, const rwkvq_desc* mu_desc,
                        const void* mu_image_dev, const void* x_fp16_dev, const void* xprev_fp16_dev,
                        int B, void* y_dev, int y_dtype, void* workspace_dev, size_t workspace_bytes,
                        void* stream);

/*
 * rwkvq_gemv without a workspace argument, for callers that must not allocate device memory:
 * code running where cudaMalloc is forbidden or unavailable (inside a pre-sized memory pool, in a
 * real-time or embedded serving loop, in a plug-in that is only handed its inputs and outputs).
 * The paper has no counterpart; this is a convenience of this library.  Inputs and outputs are
 * the caller's, exactly as for rwkvq_gemv; the split-K scratch is a fixed array of
 * rwkvq_gemv_static_max_scratch_bytes() (8 MiB) inside the library, held by every GPU that loads
 * it until the process exits.  A product whose scratch would be larger is refused with
 * RWKVQ_ENOMEM (use rwkvq_gemv with your own workspace).  The call allocates nothing, on host or
 * device.  The first call on each device looks up the array's device address (that device must be
 * current) and should therefore be made before any stream capture begins.  All calls share the
 * one array: calls that overlap on the same GPU (different streams) race on it and give wrong
 * results; issue them on one stream or separate them with events.
 */
size_t rwkvq_gemv_static_max_scratch_bytes(void);
rwkvq_status rwkvq_gemv_static(const rwkvq_desc* W_desc, const void* W_image_dev, const rwkvq_desc* mu_desc,
                               const void* mu_image_dev, const void* x_fp16_dev, const void* xprev_fp16_dev,
                               int B, void* y_dev, int y_dtype, void* stream);

/*
 * Where a product of a decode step takes its input row x[b][0..ic) from, when it is not a plain
 * fp16 buffer: the element-wise operators that sit between the projections of an RWKV block
 * (Appendix A.1).  The step computes them once per stage, after the barrier that completes the
 * stage before, in fp32, rounds x to fp16 and then applies the token-shift mix (if mu is given).
 *   RWKVQ_IN_BUFFER  x = x_fp16_dev (the plain case; every other field below is ignored).
 *   RWKVQ_IN_WKV     x = sigmoid(src) * wkv (Eq. 24) with src = r, and wkv of Eq. 23 from k_f32,
 *                    v_f32 (outputs of earlier products, [B][ic] fp32) and the running history
 *                    sums.  The sums are kept scaled by a running exponent for range:
 *                    state_a = e^{-p} * sum f(i) v_i, state_b = e^{-p} * sum f(i), state_p = p,
 *                    each [B][ic] fp32, updated in place for the next token (start a sequence
 *                    with a = b = 0, p = -1e30).  u_f32, w_f32: [ic] bonus and decay (the history
 *                    decays by e^{-w} per token).
 *   RWKVQ_IN_RELU2   x = max(src, 0)^2 (Eq. 27) with src = k'.
 *   RWKVQ_IN_F32     x = src, or sigmoid(gate_f32) * src when gate_f32 != NULL (Eq. 27: the
 *                    block's output as the next block's input), src / gate [B][ic] fp32.
 * flags & RWKVQ_INF_RMSNORM (RWKVQ_IN_F32 only, ic a multiple of 64): the row is divided by its root
 * mean square, x = v / sqrt(mean_j v[b][j]^2 + 1e-6) with v = src (* sigmoid(gate)).  The appendix
 * prints no normalisation, but a chain of its blocks does not keep its activations in range
 * without one (the squared ReLU makes magnitudes collapse or blow up within a few blocks); the
 * models the paper quantizes normalise at exactly these two places, the inputs of time mixing and
 * of channel mixing.  No learned weight or bias: use scale_f32 for a gain.
 * scale_f32 (kinds other than RWKVQ_IN_BUFFER, may be NULL): one float in device memory, read at run
 * time, that multiplies the operator's result before it is rounded to fp16.
 * xprev_out_fp16 (any kind, may be NULL): receives this token's x (before the mix), [B][ic]
 * fp16; it may be the very buffer xprev_fp16_dev points to (each element is read, then written,
 * by one thread), which makes the previous-token state advance by itself from step to step.  A
 * buffer that is updated this way must belong to ONE product.
 * All pointers are device memory, 16-byte aligned, owned by the caller.
 */
typedef enum { RWKVQ_IN_BUFFER = 0, RWKVQ_IN_WKV = 1, RWKVQ_IN_RELU2 = 2, RWKVQ_IN_F32 = 3 } rwkvq_input_kind;
#define RWKVQ_INF_RMSNORM 1   /* RWKVQ_IN_F32 only */
typedef struct {
  int32_t kind;               /* rwkvq_input_kind */
  int32_t flags;              /* RWKVQ_INF_* */
  const float* src_f32;
  const float* k_f32;
  const float* v_f32;
  float* state_a;
  float* state_b;
  float* state_p;
  const float* u_f32;
  const float* w_f32;
  const float* gate_f32;
  void* xprev_out_fp16;
  const float* scale_f32;     /* one float on the device, or NULL */
} rwkvq_input_xform;

/* One product of a decode step (same meaning as the rwkvq_gemv arguments).  `stage` orders the
 * step: every product of stage s is complete before any activation of stage s+1 is read.
 * `in` all zero = the input is x_fp16_dev; otherwise x_fp16_dev may be NULL (see above). */
typedef struct {
  rwkvq_desc W_desc;
  const void* W_image_dev;
  rwkvq_desc mu_desc;         /* ignored when mu_image_dev == NULL */
  const void* mu_image_dev;
  const void* x_fp16_dev;
  const void* xprev_fp16_dev;
  void* y_dev;
  int32_t stage;
  int32_t y_dtype;
  rwkvq_input_xform in;
} rwkvq_gemv_op;

/*
 * A whole decode step (all projections of all layers, Appendix A.1) as ONE persistent launch:
 * packed weights are streamed through shared memory continuously across products and stages
 * while a grid-wide barrier enforces the stage order.  Partial sums of a row are added into the
 * output with fp32 atomics: results are within the stated tolerance but not bit-reproducible
 * from run to run.  rwkvq_step_plan builds the schedule on
 * the host and copies it into plan_dev (rwkvq_step_plan_bytes() bytes, caller-owned); the plan
 * embeds the pointers of `ops`, so the buffers must stay where they are.  rwkvq_step_run launches
 * it.  ops must be sorted by stage (non-decreasing).  Errors as rwkvq_gemv plus ETIMEOUT through
 * rwkvq_device_status.
 */
size_t rwkvq_step_plan_bytes(const rwkvq_gemv_op* ops, int n_ops, int B);
rwkvq_status rwkvq_step_plan(const rwkvq_gemv_op* ops, int n_ops, int B, void* plan_dev,
                             size_t plan_bytes, void* stream);
rwkvq_status rwkvq_step_run(const void* plan_dev, size_t plan_bytes, void* stream);
/* Forget the host-side record of the plan written to plan_dev (call it before the buffer is freed
 * or reused for something else: the record is keyed by the buffer's address).  EINVAL if there is
 * no such plan.  Host only. */
rwkvq_status rwkvq_step_plan_release(const void* plan_dev);
/*
 * Waits inside the step kernel are bounded: a warp that has polled a barrier poll_limit times
 * (default 2^22, several seconds) gives up, the kernel returns and rwkvq_device_status reports
 * ETIMEOUT.  After an ETIMEOUT the caller must call rwkvq_device_status before the plan's next
 * rwkvq_step_run, which then clears the plan's barrier words and starts over; outputs of the run
 * that gave up are undefined.  This call sets the limit for later runs of one plan (0 = default).
 * wait_skew is added to every barrier target; any value but 0 makes every stage barrier
 * unreachable and exists so that a test can watch the waits run out.  Host only.
 */
rwkvq_status rwkvq_step_set_wait(const void* plan_dev, uint32_t poll_limit, uint32_t wait_skew);
/*
 * Host-only check of the schedule rwkvq_step_plan would build for n_ctas CTAs (no device is
 * touched; device pointers are only stored): counts_host[n_counts] receives, product after product,
 * for every 16-row slice and every 256-column tile [oc/16][ic_pad/256] how many times the schedule
 * hands that record to a consumer warp (the caller zero-fills it; a correct schedule writes 1
 * everywhere), and cta_items_host[n_ctas] (may be NULL) the records each CTA consumes.  The
 * products must have distinct y_dev.  Errors as rwkvq_step_plan_bytes, plus EINVAL for a
 * schedule that is inconsistent with itself and ENOMEM for a short counts array.
 */
rwkvq_status rwkvq_step_plan_cover(const rwkvq_gemv_op* ops, int n_ops, int B, int n_ctas,
                                   uint32_t* counts_host, size_t n_counts, uint32_t* cta_items_host);
/*
 * The same step for callers whose activations live in host memory: act_bytes are copied from act_host
 * to act_dev (the device buffer the plan's x / x_prev pointers lie in), the step runs, and y_bytes are
 * copied from y_dev (the buffer the plan's outputs lie in) to y_host.  Everything is ordered behind what
 * `stream` already holds, and `stream` ends behind all of it: the caller synchronizes `stream` before
 * reading y_host or changing act_host.  Small steps (less than 8 MB of copies) run the three parts one
 * after the other on `stream`.  Larger ones overlap them: the activations are copied in chunks of 4 MB
 * on a stream of the library's own while the step is already running (its input stages wait, bounded,
 * for the chunk that holds what they are about to read), and the outputs are copied, on another stream,
 * stage by stage as soon as the stage barrier that completes them has been passed, provided the stages'
 * outputs lie one behind the other inside [y_dev, y_dev + y_bytes) (otherwise in one piece at the end).
 * The bytes that reach y_host are those of the plain order.  Host buffers should be page-locked,
 * otherwise the copies serialize with the host.  A size of 0 skips that copy.  Calls on different
 * streams of one device are serialized by the library.  The environment variable RWKVQ_HOST_OVERLAP=0
 * (read at every call) keeps every step on the plain order.  Errors: as rwkvq_step_run, ECUDA.
 */
rwkvq_status rwkvq_step_run_host(const void* plan_dev, size_t plan_bytes, const void* act_host,
                                 void* act_dev, size_t act_bytes, const void* y_dev, void* y_host,
                                 size_t y_bytes, void* stream);

/*
 * Prefill product Y[t][i] = sum_j bf16(w_hat[i][j]) * x_mix[t][j] for M tokens, bf16 x bf16 ->
 * fp32 on the tensor cores (the dense contraction of the path: Appendix A.1, the projections of
 * Eqs. 20-22 and 24-27 applied to a whole sequence).  bf16(w_hat) is the decoded weight (the fp32 rounding
 * of s*(q-z), or the fp16 codebook entry) rounded to nearest even.  x_mix[t] = X[t] +
 * (X[t-1] - X[t]) (.) mu_hat (Eq. 20), with X[-1] = xprev0 (zeros if NULL); mu NULL = no mix.
 * X_bf16_dev: [M][ic] row-major; Y_dev: [M][oc] row-major, F32 or BF16; all device pointers,
 * 16-byte aligned, owned by the caller.  workspace_dev: rwkvq_prefill_workspace_bytes() bytes,
 * 128-byte aligned; it receives x_mix in the tensor core's operand layout and a scheduling word,
 * and must not be shared by products in flight at the same time.  The call enqueues on `stream`
 * and returns; a device-side wait that ran out shows in rwkvq_device_status (ETIMEOUT).
 * Errors: EINVAL (NULL pointer, M <= 0, mu without mu_desc, xprev0 without mu, unknown y_dtype),
 * ESHAPE (oc == 1, ic not a multiple of 8), EUNSUPPORTED (format), EALIGN, ENOMEM (workspace
 * too small), ECUDA.
 */
size_t rwkvq_prefill_workspace_bytes(const rwkvq_desc* W_desc, int M, int has_mu);
rwkvq_status rwkvq_gemm_prefill(const rwkvq_desc* W_desc, const void* W_image_dev,
                                const rwkvq_desc* mu_desc, const void* mu_image_dev,
                                const void* X_bf16_dev, const void* xprev0_bf16_dev, int M,
                                void* Y_dev, int y_dtype, void* workspace_dev,
                                size_t workspace_bytes, void* stream);
/*
 * Up to 16 independent prefill products over the same M tokens as ONE persistent launch (plus one
 * small mix launch per product): the output tiles of all products are handed to the SMs from one
 * queue, longest contraction first, so no SM idles at the end of a short product.  The products
 * of one dependency stage of a layer (R, K, V, G; or the channel-mix key and receptance) are such
 * a group.  Each entry has the arguments of rwkvq_gemm_prefill; outputs and workspaces must be
 * pairwise distinct.  Errors as rwkvq_gemm_prefill, checked for every product before anything is
 * enqueued; EUNSUPPORTED for more than 16 products; EINVAL for a shared output or workspace.
 */
typedef struct rwkvq_prefill_op {
  const rwkvq_desc* W_desc;
  const void* W_image_dev;
  const rwkvq_desc* mu_desc;      /* NULL with mu_image_dev == NULL */
  const void* mu_image_dev;
  const void* X_bf16_dev;
  const void* xprev0_bf16_dev;    /* may be NULL */
  void* Y_dev;
  void* workspace_dev;
  size_t workspace_bytes;
} rwkvq_prefill_op;
rwkvq_status rwkvq_gemm_prefill_grouped(const rwkvq_prefill_op* ops, int n_ops, int M, int y_dtype,
                                        void* stream);

/*
 * Decode the packed matrix to out_dev[oc][ic]: F32 = the exact value s*(q-z) (two IEEE fp32
 * operations: subtract, then multiply) or the fp16 codebook entry; BF16 = that value rounded to
 * nearest even.  Uses the same device unpack routines as the products (test surface for
 * "decoded weights are bit-exact").  For vectors (oc == 1) out_dev has ic elements.
 */
rwkvq_status rwkvq_dequant(const rwkvq_desc* W_desc, const void* W_image_dev, void* out_dev,
                           int dtype, void* stream);

/*
 * Description (padded sizes, image_bytes, stream_bytes) of the image that rwkvq_pack and
 * rwkvq_quantize_dev produce for an oc x ic matrix (or a vector, oc == 1 with method VQ) under
 * `cfg`; only method, bits, group, vec_dim and tile of cfg are read.  Errors as rwkvq_pack.
 */
rwkvq_status rwkvq_desc_for(const rwkvq_quant_cfg* cfg, int oc, int ic, rwkvq_desc* desc_out);

/*
 * The quantizers of rwkvq_pack as device kernels: W[oc][ic] fp16 in device memory is quantized
 * and written as a packed image straight into image_dev (256-byte aligned, at least
 * desc.image_bytes of rwkvq_desc_for), ready for every product call above.
 *  SQ (Eq. 2): codes, scales and zero points are identical to rwkvq_pack's (same rounding rules),
 *      bit for bit.
 *  VQ (Eq. 3): one thread block per 256 x 256 tile (or per vector) runs k-means++ seeding and
 *      cfg->kmeans_iters Lloyd iterations in fp32 with exact integer cluster sums, rounds the
 *      centres to fp16 and takes the final assignment in fp64 against the rounded centres (lowest
 *      index wins ties).  Random draws come from the library's generator seeded with cfg->seed and
 *      the tile number; results are reproducible but differ from rwkvq_pack's codebooks.
 *  elem_weight_dev (vectors only, else NULL): fp32 [ic], the X^2 of Section 4.2 Eq. 19 for each
 *      element of mu.  Vectors are then assigned by the weighted distance and centres move to the
 *      weighted means (fp64, fixed order), which is the weighted k-means of Section 4.2.
 *  cfg->codes_in must be NULL.  The image carries no checksum (rwkvq_image_unpack accepts that).
 *  workspace_dev: rwkvq_quantize_workspace_bytes() bytes, 16-byte aligned, contents irrelevant.
 * The call synchronizes `stream` before it returns (it reads back a flag word).  Errors: EINVAL,
 * ESHAPE, EUNSUPPORTED, EALIGN, ENOMEM (image or workspace too small), ENONFINITE, ECUDA.
 */
size_t rwkvq_quantize_workspace_bytes(void);
rwkvq_status rwkvq_quantize_dev(const void* w_fp16_dev, int oc, int ic, const rwkvq_quant_cfg* cfg,
                                const float* elem_weight_dev, void* image_dev, size_t image_bytes,
                                rwkvq_desc* desc_out, void* workspace_dev, size_t workspace_bytes,
                                void* stream);

/*
 * rwkvq_quantize_dev in two halves, for quantizing many matrices without a host round trip per
 * matrix.  rwkvq_quantize_dev_async only enqueues the kernels (same arguments and argument errors);
 * a NaN/Inf weight sets a flag in the first word of workspace_dev, which must be zero before the
 * first call and is shared by every call that uses the same workspace.  rwkvq_quantize_check
 * synchronizes `stream`, returns RWKVQ_ENONFINITE if the flag was set by any call since the last
 * check (RWKVQ_OK otherwise) and clears it.
 */
rwkvq_status rwkvq_quantize_dev_async(const void* w_fp16_dev, int oc, int ic, const rwkvq_quant_cfg* cfg,
                                      const float* elem_weight_dev, void* image_dev, size_t image_bytes,
                                      rwkvq_desc* desc_out, void* workspace_dev, size_t workspace_bytes,
                                      void* stream);
rwkvq_status rwkvq_quantize_check(void* workspace_dev, void* stream);

/*
 * Representative X of a batch of calibration activations (Section 4.2): for each of the n
 * positions, the n_samples values samples_dev[s][j] (fp32, row-major [n_samples][n],
 * 2 <= n_samples <= 1024) are limited to the range between their pct-th and (100 - pct)-th
 * percentiles (linear interpolation between order statistics, 0 <= pct < 50) and averaged in
 * fp64.  rep_dev[j] receives the mean, rep_sq_dev[j] its square (the weight of Eq. 19); either
 * may be NULL.  Asynchronous on `stream`.  Errors: EINVAL, ECUDA.
 */
rwkvq_status rwkvq_calib_representative(const float* samples_dev, int n_samples, int n, double pct,
                                        float* rep_dev, float* rep_sq_dev, void* stream);

/*
 * Quantization error of a packed matrix against the fp16 matrix it was made from:
 * *sse_host = sum over all weights of (w - w_hat)^2, accumulated in fp64 with the decode routines
 * of rwkvq_dequant (per-record sums combined in a fixed order, so the value is reproducible).
 * Comparing it between an SQ and a VQ image of the same matrix is the "MSE" selector of the
 * ablation in Section 5.3.  Matrices only.  workspace_dev: rwkvq_quant_error_workspace_bytes()
 * bytes, 16-byte aligned.  Synchronizes `stream`.  Errors: EINVAL, ESHAPE, EALIGN, ENOMEM, ECUDA.
 */
size_t rwkvq_quant_error_workspace_bytes(const rwkvq_desc* W_desc);
rwkvq_status rwkvq_quant_error(const void* w_fp16_dev, const rwkvq_desc* W_desc, const void* W_image_dev,
                               double* sse_host, void* workspace_dev, size_t workspace_bytes,
                               void* stream);

/* Device status word of the last launches on this device: RWKVQ_OK, or ETIMEOUT if a bounded
 * wait inside a kernel gave up.  Synchronizes `stream`; clears the word. */
rwkvq_status rwkvq_device_status(void* stream);
const char* rwkvq_status_str(rwkvq_status s);
/* Text of the last CUDA error seen by this thread's library calls ("" if none). */
const char* rwkvq_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* RWKVQ_H_ */
