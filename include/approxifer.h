/*
 * approxifer.h  --  C ABI of the ApproxIFER encode / decode / locate library for
 * NVIDIA B200 (sm_100a).
 *
 * The library implements the data-parallel hot path of ApproxIFER
 * (arXiv 2109.09868, Section 3): the Berrut rational-interpolation encoder,
 * the straggler-masked Berrut decoder and the Byzantine-worker locator
 * (Algorithm 2; Algorithm 1's homogeneous system and Algorithm 3's rational
 * function as alternatives), over G independent groups at a time.
 *
 * Notation.  K = queries per group (j = 0..K-1).  W = number of workers =
 * number of coded queries (i = 0..W-1); the paper counts workers 0..N, so
 * W = N+1.  E = Byzantine workers to locate.  D / C = payload elements per
 * query / per prediction.  Nodes (Section 3, "Encoding"):
 *     alpha_j = cos((2j+1) pi / (2K)),      beta_i = cos(i pi / (W-1)).
 *
 * Common rules for every entry point (the *_host variants further down take
 * HOST arrays instead and say so)
 *   - All array arguments are DEVICE pointers owned by the caller (global
 *     memory of the current device), fp32 payloads, innermost dimension
 *     contiguous; "gstride" / "rstride" are the distances, in ELEMENTS, between
 *     consecutive groups / consecutive rows of a group.  Inputs and outputs
 *     must not overlap.  `params` is a HOST pointer, read during the call.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL =
 *     the legacy default stream) and the call returns without synchronising.
 *     The library never allocates device memory (its image contains one fixed
 *     staging array, see approxifer_encode_host_static), keeps no per-call
 *     state and no setting (only immutable host-side caches: the node tables
 *     of each (K, W) seen, the current device's multiprocessor count and
 *     shared-memory size) and may be called from several host threads on
 *     different streams.
 *   - 16-byte aligned bases with D (or C) and all strides multiples of 4 take
 *     the 128-bit fast path; anything else runs a slower element-wise GPU
 *     path.  There is no CPU fallback.
 *   - Return value: APPROXIFER_OK or a negative APPROXIFER_E_* code.  Argument
 *     errors are detected on the host before anything is launched.  G == 0 is
 *     a valid no-op.
 *   - Per-group conditions are reported as APPROXIFER_ST_* bits in the
 *     optional `status[G]` output, never as a fault.
 */
#ifndef APPROXIFER_H_
#define APPROXIFER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define APPROXIFER_VERSION 100 /* major*10000 + minor*100 + patch */

#define APPROXIFER_MAX_K 32
#define APPROXIFER_MAX_W 32

/* return codes */
#define APPROXIFER_OK 0
#define APPROXIFER_E_NULL (-1)  /* a required pointer is NULL */
#define APPROXIFER_E_RANGE (-2) /* K not in 1..32, W not in 2..32, E < 0, G < 0, D < 1, D > 2^31, stride < row length */
#define APPROXIFER_E_PARAM (-3) /* locate: E < 1, 2(K+E) > W, or the homogeneous form with K+E > 13; unknown flag bits */
#define APPROXIFER_E_CUDA (-4)  /* the CUDA runtime reported an error at launch */
#define APPROXIFER_E_WORKSPACE (-5) /* host-buffer entry points: the device workspace cannot hold one group */
#define APPROXIFER_E_TOO_LARGE (-6) /* approxifer_encode_host_static: the batch does not fit the built-in staging area */

/* params.flags */
#define APPROXIFER_SIGN_RANK 0u         /* decoder sign (-1)^(rank of worker i among those used); default */
#define APPROXIFER_SIGN_WORKER_INDEX 1u /* decoder sign (-1)^i, the decoding equation read literally */
#define APPROXIFER_LOCATE_HOMOGENEOUS 2u /* locator: Algorithm 1's homogeneous system (|Q| = 1) instead of Q_0 = 1 */
#define APPROXIFER_ONE_PASS 4u           /* approxifer_locate_decode: one kernel for both steps wherever it exists */
#define APPROXIFER_TWO_LAUNCHES 8u       /* approxifer_locate_decode: always the two kernels back to back */

/* status[g] bits */
#define APPROXIFER_ST_NO_WORKERS 1u             /* decode: no worker present; the group's output is zero-filled */
#define APPROXIFER_ST_FEW_WORKERS 2u            /* decode: fewer than K workers present; computed anyway */
#define APPROXIFER_ST_LOCATE_UNDERDETERMINED 4u /* locate: fewer than 2(K+E) workers present; nothing located */
#define APPROXIFER_ST_NONFINITE 8u              /* locate: some Q(beta_i) was not finite (ranked as +inf) */
#define APPROXIFER_ST_TIMEOUT 16u               /* decode: a bounded wait on a staged copy gave up before this group was finished;
                                                   its output is unspecified (never set in a correct run) */

/*
 * One params struct serves a whole encode -> locate -> decode pipeline: every entry point reads the fields
 * that concern it and ignores the rest.  E is ignored by encode and decode.  APPROXIFER_SIGN_WORKER_INDEX
 * concerns the decoders only (approxifer_decode, approxifer_decode_host, step 2 of approxifer_locate_decode);
 * APPROXIFER_LOCATE_HOMOGENEOUS concerns the locators only (approxifer_locate, approxifer_locate_host, step 1 of
 * approxifer_locate_decode) -- approxifer_decode_rational always uses Q_0 = 1, as Algorithm 3 prints it, and the
 * encoders have no flag.  A bit that no entry point defines is APPROXIFER_E_PARAM everywhere.
 */
typedef struct approxifer_params {
  int32_t K;      /* 1..32 queries per group */
  int32_t W;      /* 2..32 workers (paper: N+1) */
  int32_t E;      /* Byzantine workers to locate; ignored by encode and decode */
  uint32_t flags; /* APPROXIFER_SIGN_* | APPROXIFER_LOCATE_* */
} approxifer_params;

/*
 * Encoder (Section 3, "ApproxIFER Encoding"):
 *     Xt[g][i][:] = u_g(beta_i) = sum_j l_j(beta_i) X[g][j][:],
 *     l_j(z) = [(-1)^j/(z-alpha_j)] / sum_k (-1)^k/(z-alpha_k).
 * If beta_i equals some alpha_j (exactly when (2j+1)(W-1) == 2Ki) the row is
 * the limit value X[g][j][:].
 *   X   in,  [G][K][D], x_rstride >= D, x_gstride >= 0 (elements)
 *   Xt  out, [G][W][D], strides xt_gstride, xt_rstride >= D; a worker-major
 *            layout [W][G][D] is expressed as xt_gstride = D, xt_rstride = G*D.
 * fp32 accumulation, one fused multiply-add per term, j ascending.
 */
int approxifer_encode(const approxifer_params* params, int64_t G, int64_t D,
                      const float* X, int64_t x_gstride, int64_t x_rstride,
                      float* Xt, int64_t xt_gstride, int64_t xt_rstride,
                      void* cuda_stream);

/*
 * Decoder (Section 3, "ApproxIFER Decoding", step 2):
 *     Yhat[g][j][:] = r_g(alpha_j),
 *     r_g(z) = sum_{i in F_g} [s_i/(z-beta_i)] Yt[g][i][:] / sum_{i in F_g} s_i/(z-beta_i),
 * F_g = workers whose bit is set in mask[g] (bits >= W are ignored), taken in
 * ascending order; s_i = (-1)^(position of i in F_g) by default, (-1)^i with
 * APPROXIFER_SIGN_WORKER_INDEX.  Every worker in the mask is used.  If
 * alpha_j equals beta_i for a present worker i, Yhat[g][j][:] = Yt[g][i][:].
 *   Yt      in,  [G][W][C]; rows of absent workers may hold anything (NaN
 *                included) and never influence the output
 *   mask    in,  [G] uint32, bit i = worker i's prediction arrived
 *   Yhat    out, [G][K][C]
 *   n_used  out, [G] int32 = |F_g|, or NULL
 *   status  out, [G] uint32 of APPROXIFER_ST_* bits, or NULL
 */
int approxifer_decode(const approxifer_params* params, int64_t G, int64_t C,
                      const float* Yt, int64_t yt_gstride, int64_t yt_rstride,
                      const uint32_t* mask,
                      float* Yhat, int64_t yh_gstride, int64_t yh_rstride,
                      int32_t* n_used, uint32_t* status, void* cuda_stream);

/*
 * The encoder and the decoder on bfloat16 payloads: the same formulas (Section 3, "ApproxIFER Encoding" and
 * "ApproxIFER Decoding", step 2), with X / Xt and Yt / Yhat holding bfloat16 elements (uint16_t bit patterns:
 * the upper half of an IEEE-754 binary32), which halves the bytes the two memory-bound kernels move.  The paper
 * fixes no storage precision; here a stored bfloat16 IS the number it denotes (widened exactly), weights and
 * sums are fp32 exactly as in the fp32 entry points, and each result is rounded once to the nearest bfloat16,
 * ties to even.  Strides are in ELEMENTS (of 2 bytes).  8-byte aligned bases with D (or C) and all strides
 * multiples of 4 take the 64-bit path, anything else an element-wise one.  Arguments, mask, n_used, status and
 * return codes as in approxifer_encode / approxifer_decode.
 */
int approxifer_encode_bf16(const approxifer_params* params, int64_t G, int64_t D,
                           const uint16_t* X, int64_t x_gstride, int64_t x_rstride,
                           uint16_t* Xt, int64_t xt_gstride, int64_t xt_rstride,
                           void* cuda_stream);
int approxifer_decode_bf16(const approxifer_params* params, int64_t G, int64_t C,
                           const uint16_t* Yt, int64_t yt_gstride, int64_t yt_rstride,
                           const uint32_t* mask,
                           uint16_t* Yhat, int64_t yh_gstride, int64_t yh_rstride,
                           int32_t* n_used, uint32_t* status, void* cuda_stream);

/*
 * Byzantine-worker locator (Algorithm 2; Algorithm 1 is its inner step; the
 * theory is Appendix A, Theorem 1).  For every group and every class c:
 * least-squares solution of
 *     P(beta_i) = Yt[g][i][c] * Q(beta_i),   i in A_avl (the mask),
 *     P(x) = sum_{k<K+E} P_k x^k,  Q(x) = 1 + sum_{1<=k<K+E} Q_k x^k,
 * a_i = Q(beta_i), the E workers with the smallest |a_i| get one vote each;
 * the E workers with the most votes over all classes are reported.  Ties, in
 * both selections, go to the lower worker index.  The solve runs in fp64.
 *   adv           out, [G][E] int32, ascending; -1 when nothing was located
 *   trusted_mask  out, [G] uint32 = mask (bits < W) minus the located workers
 *   status        out, [G] uint32 or NULL
 * Requires E >= 1 and 2(K+E) <= W.  A group with fewer than 2(K+E) workers
 * present gets adv = -1, trusted_mask = mask and ST_LOCATE_UNDERDETERMINED.
 *
 * With APPROXIFER_LOCATE_HOMOGENEOUS in params.flags the per-class step is
 * Algorithm 1 as printed (Section 3, "Rational Interpolation with Erroneous
 * Evaluations"): Q(x) = sum_{k<K+E} Q_k x^k with Q_0 free, and the homogeneous
 * system P(beta_i) = y_i Q(beta_i) is solved in the least-squares sense over
 * all P and over Q with sum_k Q_k^2 = 1 (the smallest singular direction).
 * Selection, vote, outputs and status bits are the same.  This form has no
 * special case at a node equal to 0 (odd W), where Q_0 = 1 pins a_i to 1.
 * Available for K+E <= 13; APPROXIFER_E_PARAM otherwise.
 */
int approxifer_locate(const approxifer_params* params, int64_t G, int64_t C,
                      const float* Yt, int64_t yt_gstride, int64_t yt_rstride,
                      const uint32_t* mask,
                      int32_t* adv, uint32_t* trusted_mask, uint32_t* status,
                      void* cuda_stream);

/*
 * Rational decoding (Algorithm 3, Appendix A: "BW-type rational interpolation in presence of errors").
 * For every group and class the polynomials P, Q of degree < K+E with
 *     P(beta_i) = Yt[g][i][c] * Q(beta_i),   i in the mask,   Q_0 = 1
 * are found by least squares exactly as in approxifer_locate, and instead of locating anything the rational
 * function itself is returned at the query nodes:
 *     Yhat[g][j][c] = P(alpha_j) / Q(alpha_j).
 * By the theorem that follows Algorithm 3 this equals the underlying rational function when at most E of the
 * available predictions are wrong and at least 2(K+E) are available -- for a model that is linear in its input
 * it returns the model's own predictions, not Berrut's approximation of them.  The paper warns that the division
 * is numerically fragile (it amplifies the fp32 rounding of the inputs by up to ~1e5 at K+E = 10) and uses
 * Algorithm 2 + Berrut decoding instead; this entry point is the alternative, for callers who want it.
 *   Yt, mask   as for approxifer_locate            Yhat  out, [G][K][C]
 *   status     out, [G] uint32 or NULL: ST_LOCATE_UNDERDETERMINED (fewer than 2(K+E) workers present; the
 *              group's output is zero-filled), ST_NONFINITE (some output was not finite: a root of Q at alpha_j)
 * Requires E >= 0, 2 <= K+E <= 13 and 2(K+E) <= W (APPROXIFER_E_PARAM otherwise).  The solve runs in fp64.
 */
int approxifer_decode_rational(const approxifer_params* params, int64_t G, int64_t C,
                               const float* Yt, int64_t yt_gstride, int64_t yt_rstride,
                               const uint32_t* mask,
                               float* Yhat, int64_t yh_gstride, int64_t yh_rstride,
                               uint32_t* status, void* cuda_stream);

/*
 * The decoder's two steps in one call (Section 3, "ApproxIFER Decoding", steps 1 and 2): locate the E
 * Byzantine workers of every group (Algorithm 2), then decode from the workers that are present and were
 * not located.  Equivalent, bit for bit, to approxifer_locate followed by approxifer_decode with
 * `trusted_mask` as the mask.  `trusted_mask` [G] is required (it carries the result of step 1 to step 2 on the
 * device); `adv` [G][E], `n_used` [G], `locate_status` [G] and `decode_status` [G] are as in the two entry
 * points (`adv` is required, the other three may be NULL).
 *
 * The call is either one kernel -- the locator with the decoding as its tail, available for Algorithm 2's form
 * with K+E <= 10 and C <= 128 -- or the two kernels back to back on `cuda_stream`.  One kernel saves a launch
 * and a pass over the predictions, but decodes at the locator's low occupancy: it wins on small batches
 * (K = 8, W = 24, E = 2, C = 10: 44 us against 52 us up to 1,024 groups, equal at 4,096) and loses about a tenth
 * on large ones (641 us against 591 us at 65,536 groups), so by default it is taken for batches of up to
 * APPROXIFER_ONE_PASS_MAX_GROUPS groups.  APPROXIFER_ONE_PASS / APPROXIFER_TWO_LAUNCHES in params.flags override
 * the choice (ONE_PASS where no such kernel exists still runs the two).
 */
#define APPROXIFER_ONE_PASS_MAX_GROUPS 4096
int approxifer_locate_decode(const approxifer_params* params, int64_t G, int64_t C,
                             const float* Yt, int64_t yt_gstride, int64_t yt_rstride,
                             const uint32_t* mask,
                             int32_t* adv, uint32_t* trusted_mask,
                             float* Yhat, int64_t yh_gstride, int64_t yh_rstride,
                             int32_t* n_used, uint32_t* locate_status, uint32_t* decode_status,
                             void* cuda_stream);

/*
 * Scatter / gather variants for the paper's serving architecture (Section 2, "Problem Formulation and System Model":
 * the coded query i goes to worker i, whose prediction comes back from it): every worker's batch is a buffer of
 * its own -- on this GPU, or on a peer GPU whose memory is mapped into this process -- instead of a row of one
 * array.  `Xt_rows` / `Yt_rows` are HOST arrays of W device pointers (read during the call); worker i's buffer holds
 * its row of group g at element offset g * gstride (gstride >= D or C).  The pointers must be whole elements apart;
 * 16-byte aligned buffers with D (or C) and the strides multiples of 4 take the 128-bit path.  The encoder computes
 * every coded row once and stores each to its worker's buffer; the decoder and the locator read each present
 * worker's row from its buffer.  The encoder, the locator and the decoder's per-column kernel touch these buffers
 * with plain global loads and stores only; the decoder's packed-groups kernel (dense batches of 6-10 classes, 32 MB
 * of predictions or more) reads them with bulk asynchronous copies into the issuing CTA's own shared memory (one
 * copy per worker and work item, each into one CTA's memory only).  Peer memory needs nothing but peer access
 * enabled by the caller.  Formulas, masks, outputs, status bits and return codes as in approxifer_encode / _decode / _locate;
 * APPROXIFER_E_NULL also if one of the W pointers is NULL or not a whole number of elements from the first.
 */
int approxifer_encode_scatter(const approxifer_params* params, int64_t G, int64_t D,
                              const float* X, int64_t x_gstride, int64_t x_rstride,
                              float* const* Xt_rows, int64_t xt_gstride, void* cuda_stream);
int approxifer_decode_gather(const approxifer_params* params, int64_t G, int64_t C,
                             const float* const* Yt_rows, int64_t yt_gstride, const uint32_t* mask,
                             float* Yhat, int64_t yh_gstride, int64_t yh_rstride,
                             int32_t* n_used, uint32_t* status, void* cuda_stream);
int approxifer_locate_gather(const approxifer_params* params, int64_t G, int64_t C,
                             const float* const* Yt_rows, int64_t yt_gstride, const uint32_t* mask,
                             int32_t* adv, uint32_t* trusted_mask, uint32_t* status, void* cuda_stream);

/*
 * Host-buffer variants of the three operations (same definitions and citations
 * as above).  Payloads, masks and results live in HOST memory, dense
 * ([G][K][D], [G][W][D], [G][W][C], [G][K][C], [G][E], [G]); pinned memory is
 * needed for the copies to overlap.  `workspace` is caller-owned DEVICE memory
 * of `workspace_bytes` bytes (256-byte aligned) used as staging; it is cut
 * into one slice per stream, and the batch into chunks of whole groups that
 * run as  copy in -> kernel -> copy out  on `cuda_streams[chunk % n_streams]`
 * (an array of 1..8 cudaStream_t).  With two or more streams the transfers of
 * neighbouring chunks overlap with each other and with the kernels.  The call
 * only enqueues work: host and workspace buffers must stay untouched until
 * every stream has been synchronised by the caller.  Nothing is allocated.
 * APPROXIFER_E_WORKSPACE if a slice cannot hold a single group.
 */
int approxifer_encode_host(const approxifer_params* params, int64_t G, int64_t D,
                           const float* hX, float* hXt,
                           void* workspace, size_t workspace_bytes, void* const* cuda_streams, int n_streams);
int approxifer_decode_host(const approxifer_params* params, int64_t G, int64_t C,
                           const float* hYt, const uint32_t* hmask, float* hYhat,
                           int32_t* hn_used /* or NULL */, uint32_t* hstatus /* or NULL */,
                           void* workspace, size_t workspace_bytes, void* const* cuda_streams, int n_streams);
int approxifer_locate_host(const approxifer_params* params, int64_t G, int64_t C,
                           const float* hYt, const uint32_t* hmask,
                           int32_t* hadv, uint32_t* htrusted_mask, uint32_t* hstatus /* or NULL */,
                           void* workspace, size_t workspace_bytes, void* const* cuda_streams, int n_streams);

/*
 * Encoder for callers that cannot allocate device memory.  (The paper has no
 * counterpart to this entry point; it computes exactly what approxifer_encode
 * computes.)
 *
 * Who needs it: approxifer_encode_host wants a device workspace from its
 * caller.  A front-end that shares the GPU with a model server which reserved
 * all device memory at start-up has none to hand over, and a request path that
 * must never call cudaMalloc (the call locks the device and synchronises it,
 * stalling every other stream of the process) cannot create one.  Here the
 * staging area is a fixed array of APPROXIFER_STATIC_WORKSPACE_BYTES bytes of
 * device memory that is part of the library itself: every GPU the library is
 * used on holds it from first use until the process exits.
 *
 *   hX   in,  HOST, dense [G][K][D]      hXt  out, HOST, dense [G][W][D]
 *
 * The whole batch is staged at once on `cuda_stream`: copy in, encode kernel,
 * copy out; the call only enqueues and allocates nothing (no cudaMalloc, no
 * cudaFree, no allocating library call).  With Dp = D rounded up to a multiple
 * of 4, the batch must satisfy  4*G*Dp*(K+W) (+ up to 255 bytes of alignment)
 * <= APPROXIFER_STATIC_WORKSPACE_BYTES, else APPROXIFER_E_TOO_LARGE is returned
 * and nothing is enqueued.
 *
 * The first call on each device looks up the array's device address (one
 * runtime query, no allocation) and remembers it for the life of the process;
 * make that first call before starting any stream capture on that device.
 * `cuda_stream` must belong to the device that is current during the call, and
 * the entry point must not be used again after that device has been reset
 * (cudaDeviceReset): the remembered address is not looked up a second time.  All calls on a device share the one array,
 * which keeps the previous call's bytes (nothing in it needs clearing: each
 * call overwrites what it later reads).  Two calls whose GPU work can overlap
 * -- different streams without an ordering between them, or several host
 * threads -- race on the array and corrupt each other's results; order them on
 * one stream or with events.
 */
#define APPROXIFER_STATIC_WORKSPACE_BYTES (32u << 20)
int approxifer_encode_host_static(const approxifer_params* params, int64_t G, int64_t D,
                                  const float* hX, float* hXt, void* cuda_stream);

/*
 * Test hook (not on the hot path): the weights the kernels use, computed on
 * the device by the same code.
 *   which = 0: encoder, w[W][K] = l_j(beta_i);            idx, n untouched
 *   which = 1: decoder for one `mask`, w[K][W] with columns 0..n-1 holding the
 *              weights of the n workers used (rest 0), idx[W] their indices
 *              (rest -1), *n their number (Section 3, decoding).
 * w, idx, n are device pointers.
 */
int approxifer_debug_weights(const approxifer_params* params, uint32_t mask, int which,
                             float* w, int32_t* idx, int32_t* n, void* cuda_stream);

/*
 * Test / tuning hooks (not on the hot path): approxifer_decode and approxifer_locate with the choice of kernel
 * and its launch plan given PER CALL.  The library itself keeps no such setting: these entry points change
 * nothing for any other call or thread.  Results are bit-identical for every setting (Section 3, "ApproxIFER
 * Decoding", steps 1 and 2, exactly as in the two entry points they shadow).
 *
 * `tuning` (HOST pointer, read during the call; NULL = all automatic), every field 0 = automatic:
 *   kernel       1: route the call through the per-column register-staged kernel whatever the shape; 2, 3, 4: prefer
 *                the thread-per-(query, chunk) kernel, the bulk-copy staged kernel, the packed-groups kernel where
 *                that kernel takes the shape (else the automatic choice among the remaining ones)
 *   stages       bulk-copy staged kernel (rows of >= 64 floats, 52 with K >= 8, on the 128-bit path): upper bound >= 2 on the ring depth
 *   ctas_per_sm  ... upper bound on resident CTAs per SM
 *   cols         ... 16, 32 (split 2 only), 64, 128 or 256 16-byte columns per work item (256 needs split 1 or 2
 *                and a ring that fits in shared memory, else 128 is used)
 *   split        ... 1 (K <= 16, 256 columns), 2 or 4 thread groups sharing the K queries of a column
 *   For the packed-groups kernel (dense buffers, even C <= 62) `ctas_per_sm` bounds the warps per CTA, `cols`
 *   (any positive value) the groups per work item, and `split` = 1 / 2 switches off / on the rotated word order
 *   that keeps a warp's lanes in different shared-memory banks (0: where it measured faster); `stages` is ignored
 *   (each warp's ring has two slots).
 * APPROXIFER_E_PARAM for any other value.
 *
 * Exercising the bounded waits.  The two decoders that stage predictions with asynchronous copies (bulk-copy
 * staged and packed-groups) bound every wait on such a copy and give up instead of hanging.  In a correct run
 * no wait ever runs out, so the give-up path can only be reached on purpose: `withhold_group_plus1` = g + 1
 * makes the kernel stage the work item that holds group g as usual but never announce it to the threads that
 * wait for it, and `wait_limit` (>= 65536, so that copies already started have landed long before) replaces
 * the built-in limit by that many non-blocking probes.  The waiting threads then give up after a few
 * milliseconds: the CTA (bulk-copy staged) or the warp (packed-groups) that owned the item stops, writes
 * APPROXIFER_ST_TIMEOUT into status[] of every group it has not finished (outputs of those groups are
 * unspecified), counts the event (approxifer_device_wait_timeouts) and the kernel ends normally; all other
 * groups are decoded as usual, and the context stays usable.  Nothing faults, traps or spins without limit.
 *
 * force_warp_kernel != 0 routes the locate through the warp-per-group kernel, which otherwise serves only
 * K+E > 15 (smaller K+E use the thread-per-class kernel).  Both follow Algorithm 2 and return the same sets.
 */
typedef struct approxifer_decode_tuning {
  int32_t kernel, stages, ctas_per_sm, cols, split;
  uint32_t wait_limit;          /* see below; 0 = the built-in limit */
  int64_t withhold_group_plus1; /* see below; 0 = none */
} approxifer_decode_tuning;
int approxifer_debug_decode(const approxifer_params* params, int64_t G, int64_t C,
                            const float* Yt, int64_t yt_gstride, int64_t yt_rstride,
                            const uint32_t* mask,
                            float* Yhat, int64_t yh_gstride, int64_t yh_rstride,
                            int32_t* n_used, uint32_t* status,
                            const approxifer_decode_tuning* tuning, void* cuda_stream);
int approxifer_debug_locate(const approxifer_params* params, int64_t G, int64_t C,
                            const float* Yt, int64_t yt_gstride, int64_t yt_rstride,
                            const uint32_t* mask,
                            int32_t* adv, uint32_t* trusted_mask, uint32_t* status,
                            int force_warp_kernel, void* cuda_stream);

/*
 * Host-side planning hook (no device call; the paper has no counterpart).  The packed-groups decoder keeps the
 * predictions of several consecutive groups in shared memory exactly as they lie in device memory, so groups can
 * start in the same banks; where that costs, some groups of a work item take the words of their rows in an
 * order rotated by one.  Which ones is decided on the host from a model of the bank rules (a 64-bit load costs
 * the largest number of different words that meet in one bank over the warp; a store the same per half-warp).
 * For the shape (K, W, C) this returns the groups per work item (0: the kernel does not take the shape), the
 * rotated groups as a bit set (bit s = group s of the item), and the model's count of shared-memory passes per
 * item for the loads of the worker loop plus the stores of the results, without any rotation and with the chosen
 * one (both 0 where rows are shared by several lanes and no rotation applies).  mode: 0 as the decoder decides,
 * 1 never rotate, 2 rotate whenever the model prefers a set.  All pointers HOST, all required.
 * APPROXIFER_E_PARAM for a null pointer or parameters outside 1 <= K <= W <= 32, C >= 1, mode in 0..2.
 */
int approxifer_debug_pack_rotation(int32_t K, int32_t W, int64_t C, int32_t mode, int32_t* groups_per_item,
                                   uint32_t* rotated_groups, int32_t* passes_plain, int32_t* passes_chosen);

/*
 * Measuring hook (not on the hot path; the paper has no counterpart): `blocks` CTAs of 256 threads each run
 * `iters` rounds of 64 dependent-chain-free fp32 multiply-adds per thread on registers only (16 independent
 * chains), 2 * 64 * iters * 256 * blocks flop in all.  Timed by the caller, it gives the issue rate of the plain
 * fp32 pipe -- the second roof, next to HBM bandwidth, of the skinny weighted sums of Section 3 (2 K W / (4 (K + W))
 * flop per payload byte).  `sink` is a device float that is never written in practice.
 */
int approxifer_debug_fma_peak(int iters, int blocks, float* sink, void* cuda_stream);

/*
 * Every wait on an asynchronous copy inside the kernels is bounded.  Returns how
 * many such waits have given up on the current device since the library was
 * loaded or the counter was last reset (0 in a correct run; the affected groups
 * carry APPROXIFER_ST_TIMEOUT in status[] and their outputs are unspecified), or
 * -1 if the counter cannot be read.  Synchronises the device.
 * approxifer_reset_device_wait_timeouts sets the counter back to 0.
 */
int64_t approxifer_device_wait_timeouts(void);
int approxifer_reset_device_wait_timeouts(void);

/* Human-readable text for a return code (static storage). */
const char* approxifer_strerror(int code);

/* APPROXIFER_VERSION of the loaded library. */
int approxifer_version(void);

/* Number of kernels this library has launched in this process so far. */
int64_t approxifer_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* APPROXIFER_H_ */
