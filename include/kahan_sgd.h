/*
 * kahan_sgd.h - C ABI of the lazy update (SGD with Kahan summation) in dynamic
 * fixed-point, arXiv 1810.05486, Section 2, Eq. 1 and Algorithm 1.
 *
 * Number system (Section 2, Fig. 1).  A tensor is an array of signed integer
 * mantissas sharing one exponent: value = Q * 2^e.  A parameter tensor theta has
 * m-bit mantissas (m = 8 or 16) at exponent exp_theta.  The accumulator of
 * Algorithm 1 is kept negated as the compensation c = -acc: n-bit mantissas
 * (n = 8 or 16; n = 0 selects plain low-precision SGD, Eq. 1) at exponent
 * exp_theta - s, with s = n - 1 - overlap_k, so that theta + c carries
 * m + n - 2 - overlap_k magnitude bits (Section 2).
 *
 * One step, per element (Algorithm 1, statements 1-4, c = -acc):
 *   d      = clamp(rne(g * (lr * 2^-(e_out - s))), +-2^30)   one binary32 multiply; NaN -> 0
 *   T      = theta + c - d          exact, on the finer of the input and output c grids
 *   P      = rne(T / 2^e_out)       Q_theta' = clamp(P,  +-(2^(m-1) - 1))
 *   Rq     = rne((T - Q_theta' * 2^e_out) / 2^(e_out - s))
 *                                   Q_c'     = clamp(Rq, +-(2^(n-1) - 1))
 * rne = round to nearest, ties to even.  A step reads mantissas stored at exponent
 * exp_cur and writes them at exp_next (|exp_next - exp_cur| <= 8); in the same pass it
 * reduces, per tensor, amax_theta = max |P| and amax_comp = max min(|Rq|, 2^31 - 1)
 * and counts clamped parameter mantissas, clamped compensation mantissas and
 * non-finite gradients.  After the pass, per tensor (max scan, Section 5):
 *   exp_cur <- exp_next;  exp_next <- tight fit of amax_theta (KSGD_EXP_AMAX)
 *   or unchanged (KSGD_EXP_FIXED).  Tight fit: the smallest exponent change that puts
 *   the largest mantissa in (QMAX/2, QMAX], limited to 8 binades per step and to
 *   [-64, 64]; amax_theta == 0 keeps the exponent.
 *
 * Conventions for every entry point:
 *   - "device" pointers are CUDA device memory of the current device, "host" pointers
 *     ordinary host memory.  The caller owns every buffer it passes, including the
 *     workspace; the library owns only the host-side handle.  Except where an entry
 *     point says otherwise the library allocates and frees no device memory.
 *   - All work is enqueued on the stream given to kahan_sgd_init; nothing touches the
 *     default stream.  Only kahan_sgd_init, kahan_sgd_amax, kahan_sgd_step_host and
 *     kahan_sgd_destroy wait for the stream.
 *   - Return value 0 = success, negative = one of the KSGD_ERR_* codes.  No entry
 *     point throws, aborts or traps on the device.  Saturation and non-finite
 *     gradients are data, not errors: they are counted.
 */
#ifndef KAHAN_SGD_H_
#define KAHAN_SGD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ksgd_handle ksgd_handle; /* opaque, host memory, library-owned */

typedef struct {
  void*   theta;          /* device, int8_t[numel] (theta_bits 8) or int16_t[numel] (16); in place; 16-byte aligned */
  void*   comp;           /* device, int8_t/int16_t[numel] by comp_bits; in place; 16-byte aligned; NULL iff comp_bits == 0 */
  int64_t numel;          /* > 0 */
  int32_t theta_bits;     /* 8 | 16 */
  int32_t comp_bits;      /* 0 (plain SGD, Eq. 1) | 8 | 16 */
  int32_t overlap_k;      /* 0 .. comp_bits-1; bits of c that overlap theta; ignored when comp_bits == 0 */
  int32_t exp_theta;      /* exponent of the mantissas now stored, in [-64, 64] */
  int32_t exp_theta_next; /* exponent the first step writes (== exp_theta for a fresh start), in [-64, 64], within 8 of exp_theta */
} ksgd_tensor_desc;

typedef enum { KSGD_EXP_FIXED = 0, KSGD_EXP_AMAX = 1 } ksgd_exp_mode;

enum {
  KSGD_OK = 0,
  KSGD_ERR_NULL = -1,      /* a required pointer is NULL (or comp is non-NULL with comp_bits == 0) */
  KSGD_ERR_BITS = -2,      /* theta_bits / comp_bits not in the supported set */
  KSGD_ERR_OVERLAP = -3,   /* overlap_k outside 0 .. comp_bits-1 */
  KSGD_ERR_EXP_RANGE = -4, /* an exponent outside [-64, 64] or a first-step change larger than 8 */
  KSGD_ERR_NUMEL = -5,     /* numel <= 0, n_tensors <= 0, or more than 2^31-1 chunks in total */
  KSGD_ERR_ALIGN = -6,     /* a device pointer is not 16-byte aligned (workspace: 256) */
  KSGD_ERR_WORKSPACE = -7, /* workspace smaller than kahan_sgd_workspace_bytes */
  KSGD_ERR_LR = -8,        /* a learning rate is not finite or not > 0 */
  KSGD_ERR_CUDA = -9,      /* a CUDA runtime call failed; kahan_sgd_last_cuda_error() has its text */
  KSGD_ERR_MODE = -10,     /* exponent mode not one of ksgd_exp_mode */
  KSGD_ERR_DEVICE = -11    /* a bounded wait inside a kernel ran out (reported by kahan_sgd_amax); the step's results are invalid */
};

/*
 * Bytes of device workspace kahan_sgd_init needs for this tensor list (per-tensor
 * exponents, max-scan scratch, counters, per-step arguments and the tables that cut
 * the ragged list into tiles: about 8 bytes per 8192 elements, 170 bytes per tensor and
 * 8 to 16 KB that do not depend on the list).  Host-only computation.  Returns 0 if the
 * list is invalid (kahan_sgd_init reports why).  A tensor may have up to 2^40 elements.
 */
size_t kahan_sgd_workspace_bytes(const ksgd_tensor_desc* descs, int32_t n_tensors);

/*
 * Byte offset, inside the workspace of this list, of the 4-byte word in which a kernel
 * records the first bounded wait that ran out (0 = none; the word is sticky and
 * kahan_sgd_amax turns a non-zero value into KSGD_ERR_DEVICE).  For diagnostics, and for
 * tests of the caller's error handling that set the word from the host instead of making a
 * GPU wait run out.  Host-only computation; (size_t)-1 if the list is invalid.  (No
 * counterpart in the paper: part of the error behaviour of this boundary.)
 */
size_t kahan_sgd_workspace_error_offset(const ksgd_tensor_desc* descs, int32_t n_tensors);

/*
 * The tile table kahan_sgd_init would build for this list on a device with `sms`
 * multiprocessors (0: whole tiles only), for diagnostics and tests: how a step cuts the ragged
 * list into the pieces its blocks take in turn (block b takes entries b, b + sms, ...).
 * which: 0 = the table of ordinary steps, 1 = the table of steps on 8-bit gradients (0
 * entries for lists too short to have one).  out: host array of 3 * capacity values, or NULL
 * to count only; entry i is out[3i] = tensor, out[3i+1] = first element, out[3i+2] = number
 * of elements.  Returns the number of entries of the table (which may exceed capacity; only
 * capacity entries are written), or a negative error code for an invalid list or argument.
 * Host-only computation.  (No counterpart in the paper: the partition is this library's.)
 */
int64_t kahan_sgd_tile_table(const ksgd_tensor_desc* descs, int32_t n_tensors, int32_t sms, int32_t which,
                             int64_t* out, int64_t capacity);

/*
 * Validate the list, lay out the workspace and copy the chunk table and initial
 * exponents to it.  descs: host array of n_tensors entries, copied.  workspace: device,
 * caller-owned, at least kahan_sgd_workspace_bytes, 256-byte aligned; it must stay
 * valid and untouched by the caller until kahan_sgd_destroy.  cuda_stream: the
 * cudaStream_t (as void*) all later work is enqueued on; NULL = the legacy default
 * stream.  Waits for its copies to finish.  On error *out is NULL.
 * Ordering: the library orders its work on cuda_stream only.  Whatever the caller still
 * has in flight on another stream that writes the workspace, theta, comp or the gradients
 * (a zero-fill of a fresh allocation, an upload) must have finished, or be ordered before
 * cuda_stream by an event, when this call and the later steps are made.
 * (State of Algorithm 1: "Require theta, ..., previous theta, previous acc".)
 */
int kahan_sgd_init(ksgd_handle** out, const ksgd_tensor_desc* descs, int32_t n_tensors,
                   ksgd_exp_mode mode, void* workspace, size_t workspace_bytes,
                   void* cuda_stream);

/*
 * One lazy-update step of every tensor (Algorithm 1; Eq. 1 for comp_bits == 0), the
 * fused max scans and the exponent choice for the next step.  grads: host array of
 * n_tensors device pointers, each fp32[numel], 16-byte aligned, read-only, may change
 * from step to step.  lrs: host array of n_tensors learning rates (eta), finite and
 * > 0.  Both host arrays are consumed before the call returns.  Only enqueues work
 * (no host synchronisation).  theta and comp are updated in place.
 */
int kahan_sgd_step(ksgd_handle* h, const float* const* grads, const float* lrs);

/*
 * The same step with the gradients given as dynamic fixed-point tensors, as the paper's
 * 8-bit hardware model produces them (Section 1: every tensor of the training pass, the
 * gradients included, is INT8 or INT16 with a shared exponent; Section 4.2: INT16 gradients
 * before the last layer of AlexNet).  grads[i]: device, int8_t[numel] (grad_bits 8) or
 * int16_t[numel] (16), 16-byte aligned, read only; exp_grad[i]: host array, the exponent of
 * tensor i's gradient mantissas, in [-64, 64] (else KSGD_ERR_EXP_RANGE).  A gradient
 * Q_g * 2^exp_grad is exact in binary32, and the step is by definition the plain step on
 * that binary32 value: d = clamp(rne(fl32((Q_g * 2^exp_grad) * fl32(eta * 2^-(e_out - s)))));
 * everything else as kahan_sgd_step.  Fixed-point gradients can be made from binary32
 * ones with kahan_sgd_import (comp_bits 0, KSGD_EXP_AUTO picks the exponent from the
 * maximum).  The gradient stream shrinks from 4 bytes per parameter to 1 or 2.  Steps on
 * 8-bit gradients of long lists walk a tile table of their own, with tiles twice as large
 * (it is part of the workspace that kahan_sgd_workspace_bytes sizes and
 * kahan_sgd_init fills); which table a step uses changes no result, and steps of either kind
 * may follow one another on one handle.
 */
int kahan_sgd_step_qgrad(ksgd_handle* h, const void* const* grads, int32_t grad_bits, const int32_t* exp_grad,
                         const float* lrs);

/*
 * The same with the gradients' exponents in device memory: exp_grad_dev is a device array of
 * n_tensors int32 (4-byte aligned) that the step reads when it runs, so that exponents chosen
 * on the device by kahan_sgd_import_dev (Section 5: the exponent from a max scan) reach the
 * step without a host round trip; values outside [-64, 64] are clamped into the range.  The
 * array must stay valid and unchanged until the step has run.
 */
int kahan_sgd_step_qgrad_dev(ksgd_handle* h, const void* const* grads, int32_t grad_bits,
                             const int32_t* exp_grad_dev, const float* lrs);

/*
 * The same step for callers whose tensors live in host memory: copies each tensor's
 * theta, comp and gradient from host to the device buffers named in the descs (and to
 * grad_staging), runs the step, copies theta and comp back and waits.  theta_host /
 * comp_host / grads_host: host arrays of n_tensors host pointers (comp_host[t] ignored
 * when comp_bits == 0); page-locked memory makes the copies asynchronous.  The list is
 * processed as a pipeline of groups of neighbouring tensors (about 256 MB each): copies
 * to the device, the update, and copies back overlap, on two copy streams the handle
 * creates on first use.  The exponents of a tensor are chosen when its group is done.
 * grad_staging: device, 16-byte aligned, at least 4 * sum(round_up(numel, 4)) bytes,
 * caller-owned.
 */
int kahan_sgd_step_host(ksgd_handle* h, void* const* theta_host, void* const* comp_host,
                        const float* const* grads_host, const float* lrs,
                        void* grad_staging, size_t grad_staging_bytes);

/*
 * Results of the most recent step, per tensor (each output: host array of n_tensors
 * entries, or NULL to skip): amax_theta = max |P| and amax_comp = max |Rq| of that step
 * (Section 5 max scan); exp_theta_cur = exponent of the mantissas now in memory;
 * exp_theta_next = exponent the next step will write; n_sat_theta / n_sat_comp /
 * n_nonfinite = cumulative counts since init.  Waits for the stream.
 */
int kahan_sgd_amax(ksgd_handle* h, uint32_t* amax_theta, uint32_t* amax_comp,
                   int32_t* exp_theta_cur, int32_t* exp_theta_next,
                   uint64_t* n_sat_theta, uint64_t* n_sat_comp, uint64_t* n_nonfinite);

/*
 * Override the exponents the next step writes (host array of n_tensors entries, each in
 * [-64, 64]).  On the device each is limited to within 8 of the tensor's current
 * exponent.  Enqueues only.  (Dynamic fixed-point, Section 1: the shared exponent is
 * the caller's to steer when it knows better than the max scan.)
 */
int kahan_sgd_set_exponents(ksgd_handle* h, const int32_t* exp_theta_next);

/*
 * One step for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this entry point exists for the sake of the calling environment, not of the method.)
 *
 * kahan_sgd_init needs a device workspace from its caller, and some callers have no way to
 * get one at the moment they need it: a plug-in running inside a host program that has
 * already handed all device memory to its own pool and forbids further cudaMalloc calls;
 * a latency-critical loop where cudaMalloc's device-wide synchronisation is unacceptable.
 * For them the same scratch (exponents, max-scan slots,
 * counters, tile table) lives in a fixed array of KSGD_STATIC_SCRATCH_BYTES inside the
 * library's device image, which every GPU that loads the library holds until the process
 * exits.  The call allocates and frees no device memory, directly or through any library.
 *
 * The call is self-contained: it runs exactly one step of the whole list (same kernel,
 * same arithmetic, same results bit for bit as kahan_sgd_init + kahan_sgd_step +
 * kahan_sgd_amax on a fresh handle) and waits for it.  descs carries the state a caller
 * keeps between steps: theta/comp device pointers (updated in place), formats, and the
 * exponents exp_theta (of the stored mantissas) and exp_theta_next (to write); feed the
 * returned exp_theta_cur / exp_theta_next back into the next call's descs.  grads, lrs:
 * as for kahan_sgd_step.  Outputs (host arrays of n_tensors entries, NULL to skip): as for
 * kahan_sgd_amax, except that the three counters count this call only.
 *
 * Limits: n_tensors <= KSGD_STATIC_MAX_TENSORS and the tile table must fit the array
 * (sum over tensors of ceil(numel / 8192) tiles, 8 bytes each, plus about 100 bytes per
 * tensor: roughly 1.9e8 parameters); beyond that the call returns KSGD_ERR_WORKSPACE and
 * does nothing.
 *
 * The first call on each device looks up the array's device address and sets a kernel
 * attribute; make that first call before any stream capture begins.  Every call takes the
 * array, the SM count and the L2 size of the device that is current when it is made:
 * the device that owns cuda_stream must be current on every call, not just the first.
 * Every call copies to and from pageable host memory and waits for the stream, so the call
 * itself synchronises and cannot be part of a stream capture.  All calls on a device share
 * the one array and each call rewrites all of it, so two calls whose work overlaps on the
 * GPU (different streams, different threads) race: callers serialise them.  The list is
 * always cut into tiles of 8192 elements (the workspace path takes 16384-element tiles for
 * long lists of 8-bit tensors, and twice its usual sizes in steps on 8-bit gradients), which
 * changes no result.
 */
#define KSGD_STATIC_SCRATCH_BYTES (192 * 1024)
#define KSGD_STATIC_MAX_TENSORS 256
int kahan_sgd_step_static(const ksgd_tensor_desc* descs, int32_t n_tensors, ksgd_exp_mode mode,
                          const float* const* grads, const float* lrs, uint32_t* amax_theta,
                          uint32_t* amax_comp, int32_t* exp_theta_cur, int32_t* exp_theta_next,
                          uint64_t* n_sat_theta, uint64_t* n_sat_comp, uint64_t* n_nonfinite,
                          void* cuda_stream);

/*
 * Strict Algorithm 1 (Section 2, Algorithm 1 and Figure 1, read literally for the paper's
 * hardware model): every statement rounds into the stored format, and the accumulator is
 * an n-bit dynamic fixed-point tensor of its own whose exponent follows its own maximum
 * (Section 5), so that the overlap k of Figure 1 is a result, k = n - 1 - (e - e_acc), not
 * a parameter.  The ordinary entry points keep the sum theta + c - eta*g wide inside a step
 * and tie c's exponent to theta's; this mode exists to measure what that buys.  As
 * everywhere the tensor stored is c = -acc.  Per element, with f the smallest of the four
 * exponents (theta's and c's, read at *_in, written at *_out):
 *     d    = clamp(rne(fl32(g * fl32(eta * 2^-ec_out))), +-2^30)
 *     C1   = rne((Q_c*2^(ec_in-f) - d*2^(ec_out-f)) / 2^(ec_out-f)),  Q_c1 = clamp(C1, +-QMAX_n)
 *     T    = Q_theta*2^(e_in-f) + Q_c1*2^(ec_out-f),  P = rne(T / 2^(e_out-f)),  Q_theta' = clamp(P, +-QMAX_m)
 *     C2   = rne((T - Q_theta'*2^(e_out-f)) / 2^(ec_out-f)),  Q_c' = clamp(C2, +-QMAX_n)
 * amax_comp = max(|C1|, |C2|) and n_sat_comp counts both clamps.  c's next exponent is the
 * tight fit of amax_comp (8 binades finer when amax_comp is 0: every increment rounded away
 * or none came), kept within [e_next - 36, e_next + 8] of theta's next exponent.
 * kahan_sgd_strict_init: as kahan_sgd_init, plus exp_comp / exp_comp_next (host arrays, one
 * per tensor: c's exponent now stored and the one the first step writes; exp_comp_next NULL
 * = the same).  Every tensor needs comp_bits != 0 (else KSGD_ERR_BITS); overlap_k is
 * ignored; exponents outside [-64, 64] or outside the window above, or a first-step change
 * of c's exponent of more than 16 (the most the rule above ever asks for: 8 of its own fit
 * plus 8 of theta's move; the 64-bit sums of a step are only guaranteed up to there), give
 * KSGD_ERR_EXP_RANGE.  Both pairs are checked against their own window: (exp_theta,
 * exp_comp) and (exp_theta_next, exp_comp_next); a state read from a running handle with
 * kahan_sgd_amax and kahan_sgd_strict_exponents satisfies both, so it can be resumed.
 * kahan_sgd_strict_workspace_bytes: the size for such a list, 0 if the list or a stored
 * exponent pair is invalid (it does not see the first step's exponents and does not check them).
 * The handle then works with kahan_sgd_step, kahan_sgd_step_qgrad, kahan_sgd_amax and
 * kahan_sgd_destroy; kahan_sgd_step_host, kahan_sgd_set_exponents and
 * kahan_sgd_strict_exponents on the wrong kind of handle return KSGD_ERR_MODE.
 * kahan_sgd_strict_exponents copies c's exponents (stored / next) to the non-NULL host
 * arrays and waits for the stream.
 */
size_t kahan_sgd_strict_workspace_bytes(const ksgd_tensor_desc* descs, const int32_t* exp_comp,
                                        int32_t n_tensors);
int kahan_sgd_strict_init(ksgd_handle** out, const ksgd_tensor_desc* descs, const int32_t* exp_comp,
                          const int32_t* exp_comp_next, int32_t n_tensors, ksgd_exp_mode mode,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);
int kahan_sgd_strict_exponents(ksgd_handle* h, int32_t* exp_comp_cur, int32_t* exp_comp_next);

/* Free the host-side handle (waits for the stream first).  Device buffers stay the caller's. */
int kahan_sgd_destroy(ksgd_handle* h);

/*
 * Momentum optimizer with the lazy update (Section 4: Algorithm 1 "was implemented in the
 * optimizers"; momentum mu = 0.9 kept in INT8, INT16 for AlexNet).  The paper prints no
 * formulas for it; the form implemented is
 *     v <- mu*v + eta*g ,   theta <- theta - v   (the subtraction through Algorithm 1)
 * with the velocity v a third dynamic fixed-point tensor: mom_bits-bit mantissas with their
 * own shared exponent, which follows the max scan of |V| like theta's exponent follows
 * |P| (one step of delay, at most 8 binades per step, [-64, 64]) but with a dead band: it
 * is kept while the largest velocity mantissa stays in (QMAX/4, QMAX] and otherwise takes
 * the tight fit, because the velocity's maximum moves with every gradient.  Per element:
 *     y  = fma32(fl32(mu * 2^(ev_in - ev_out)), Q_v, fl32(g * fl32(eta * 2^-ev_out)))
 *     V  = clamp(rne(y), +-2^30), NaN -> 0 ;   Q_v' = clamp(V, +-(2^(mom_bits-1) - 1))
 *     d  = Q_v' * 2^k if k >= 0 (clamped to +-2^30), rne(Q_v' / 2^-k) otherwise,
 *          k = ev_out - (e_out - s): the stored velocity on the compensation grid
 *     then T, P, Q_theta', Rq, Q_c' as in the plain step with this d.
 * The tensor descriptions are the same ksgd_tensor_desc (comp_bits must be 8 or 16) plus
 * one ksgd_momentum_desc per tensor.  Ownership, streams,
 * return codes and the meaning of the common outputs are as for the plain entry points;
 * mus: host array of momentum coefficients, finite and >= 0 (an invalid one gives
 * KSGD_ERR_LR).  amax_mom = max |V| of the last step, n_sat_mom = clamped velocity
 * mantissas since init.
 */
typedef struct ksgd_momentum_handle ksgd_momentum_handle;

typedef struct {
  void*   mom;           /* device, int8_t[numel] (mom_bits 8) or int16_t[numel] (16); in place; 16-byte aligned */
  int32_t mom_bits;      /* 8 | 16 */
  int32_t exp_mom;       /* exponent of the velocity mantissas now stored, in [-64, 64] */
  int32_t exp_mom_next;  /* exponent the first step writes, within 8 of exp_mom */
  int32_t reserved;      /* 0 */
} ksgd_momentum_desc;

size_t kahan_sgd_momentum_workspace_bytes(const ksgd_tensor_desc* descs, const ksgd_momentum_desc* mdescs,
                                          int32_t n_tensors);
int kahan_sgd_momentum_init(ksgd_momentum_handle** out, const ksgd_tensor_desc* descs,
                            const ksgd_momentum_desc* mdescs, int32_t n_tensors, ksgd_exp_mode mode,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);
int kahan_sgd_momentum_step(ksgd_momentum_handle* h, const float* const* grads, const float* lrs,
                            const float* mus);
int kahan_sgd_momentum_amax(ksgd_momentum_handle* h, uint32_t* amax_theta, uint32_t* amax_comp,
                            uint32_t* amax_mom, int32_t* exp_theta_cur, int32_t* exp_theta_next,
                            int32_t* exp_mom_cur, int32_t* exp_mom_next, uint64_t* n_sat_theta,
                            uint64_t* n_sat_comp, uint64_t* n_sat_mom, uint64_t* n_nonfinite);
int kahan_sgd_momentum_destroy(ksgd_momentum_handle* h);

/*
 * ADAM with the lazy update (Section 4: Algorithm 1 in the optimizers; the experiments use
 * ADAM with beta1 = 0.9, beta2 = 0.999, and with beta1 = 0.5, beta2 = 0.9, eps = 1e-3; INT16
 * is needed for it because of beta2).  The paper prints no formulas for it; the form
 * implemented is the published ADAM with the bias correction folded into the step size by
 * the caller, lr_t = eta * sqrt(1 - beta2^t) / (1 - beta1^t):
 *     m <- beta1*m + (1-beta1)*g ,  v <- beta2*v + (1-beta2)*g^2 ,
 *     theta <- theta - lr_t * m / (sqrt(v) + eps)     (the subtraction through Algorithm 1)
 * with m and v two more dynamic fixed-point tensors of 16-bit mantissas, each with its own
 * shared exponent that follows the max scan of its mantissas like the momentum velocity's
 * (one step of delay, at most 8 binades per step, [-64, 64], dead band (QMAX/4, QMAX]).
 * Per element, every fl32/fma32/sqrt32/div32 one correctly rounded binary32 operation:
 *     ym = fma32(fl32(beta1 * 2^(em_in-em_out)), Q_m, fl32(g * fl32(fl32(1-beta1) * 2^-em_out)))
 *     yv = fma32(fl32(beta2 * 2^(ev_in-ev_out)), Q_v, fl32(fl32(g*g) * fl32(fl32(1-beta2) * 2^-ev_out)))
 *     M, V = clamp(rne(y), +-2^30), NaN -> 0 ;  Q_m', Q_v' = clamp(., +-32767)
 *     q  = div32(Q_m' * 2^em_out, fl32(sqrt32(max(Q_v', 1) * 2^ev_out) + eps))
 *     d  = clamp(rne(fl32(q * fl32(lr_t * 2^-(e_out - s)))), +-2^30), NaN -> 0
 *     then T, P, Q_theta', Rq, Q_c' as in the plain step with this d.
 * A second moment below the resolution of its grid is taken as one unit of the grid, not as
 * zero (which would leave eps alone in the denominator and make the step m/eps): the step of
 * such an element is bounded by |m| / sqrt(2^ev_out).  The tensor descriptions are the same
 * ksgd_tensor_desc (comp_bits must be 8 or 16) plus one ksgd_adam_desc per tensor.
 * Ownership, streams and return codes are as for the plain entry points.  lrs: host array of lr_t per tensor, finite and > 0; beta1, beta2 in [0, 1], eps
 * finite and >= 0 (otherwise KSGD_ERR_LR).  kahan_sgd_adam_amax fills the non-NULL host
 * arrays of ksgd_adam_stats (n_tensors entries each): maxima of |P|, |Rq|, |M|, |V| of the
 * last step, the exponents now stored and those the next step writes, and the counts of
 * clamped mantissas and non-finite gradients since init.
 */
typedef struct ksgd_adam_handle ksgd_adam_handle;

typedef struct {
  void*   mom1;          /* device, int16_t[numel], first moment m; in place; 16-byte aligned */
  void*   mom2;          /* device, int16_t[numel], second moment v; in place; 16-byte aligned */
  int32_t exp_m;         /* exponent of the first-moment mantissas now stored, in [-64, 64] */
  int32_t exp_m_next;    /* exponent the first step writes, within 8 of exp_m */
  int32_t exp_v;         /* the same for the second moment */
  int32_t exp_v_next;
} ksgd_adam_desc;

typedef struct {
  uint32_t *amax_theta, *amax_comp, *amax_m, *amax_v;
  int32_t  *exp_theta_cur, *exp_theta_next, *exp_m_cur, *exp_m_next, *exp_v_cur, *exp_v_next;
  uint64_t *n_sat_theta, *n_sat_comp, *n_sat_m, *n_sat_v, *n_nonfinite;
} ksgd_adam_stats;

size_t kahan_sgd_adam_workspace_bytes(const ksgd_tensor_desc* descs, const ksgd_adam_desc* adescs,
                                      int32_t n_tensors);
int kahan_sgd_adam_init(ksgd_adam_handle** out, const ksgd_tensor_desc* descs, const ksgd_adam_desc* adescs,
                        int32_t n_tensors, ksgd_exp_mode mode, void* workspace, size_t workspace_bytes,
                        void* cuda_stream);
int kahan_sgd_adam_step(ksgd_adam_handle* h, const float* const* grads, const float* lrs, float beta1,
                        float beta2, float eps);
int kahan_sgd_adam_amax(ksgd_adam_handle* h, const ksgd_adam_stats* out);
int kahan_sgd_adam_destroy(ksgd_adam_handle* h);

/*
 * Self-check of the ADAM kernel's arithmetic (no counterpart in the paper).  The kernel's
 * fast path computes sqrt32 and div32 above with short branch-free sequences instead of the
 * general correctly rounded operations; this call compares the two on the device for every
 * operand the fast path can meet -- all (Q_m', significand of the denominator) pairs at
 * eight exponent pairs including the corners of the exponent ranges (2.2e12 divisions), and
 * all Q_v' * 2^ev (4.2e6 square roots) -- and returns the numbers of differing results in
 * the two host words (both must be 0).  Takes about two seconds of GPU time; allocates
 * nothing; runs on cuda_stream and waits for it.
 */
int kahan_sgd_adam_selfcheck(uint64_t* div_mismatches, uint64_t* sqrt_mismatches, void* cuda_stream);

/*
 * fp32 -> dynamic fixed-point (Section 1: uniform linear quantization, one shared exponent
 * per tensor; Section 5: the exponent from a scan of the maximum).  src: device,
 * fp32[numel].  theta / comp: device outputs in the formats of ksgd_tensor_desc (comp NULL
 * iff comp_bits == 0).  Q_theta = clamp(rne(x / 2^e)); with a compensation tensor the part
 * theta cannot hold goes there, Q_c = clamp(rne((x - Q_theta*2^e) / 2^(e-s))), so that an
 * imported weight keeps m+n-2-k bits; NaN -> 0, +-Inf -> +-QMAX.  exp_theta: the exponent
 * to use, in [-64, 64], or KSGD_EXP_AUTO for the smallest exponent whose grid holds the
 * largest finite |x| (0 for an all-zero tensor); with KSGD_EXP_AUTO the call runs a max
 * scan whose last block picks the exponent on the device, then the quantization, which reads
 * it from device memory, and waits only to hand the exponent back; scratch: device, at least
 * 16 bytes, 4-byte aligned (cleared by the call).  *exp_theta_out (host, may be NULL)
 * receives the exponent used.  With a given exponent the call only enqueues.
 * 16-byte aligned src and 4-byte (8-bit) or 8-byte (16-bit) aligned outputs take the fast path
 * (four elements per access); anything else is converted element by element.
 *
 * kahan_sgd_import_dev: the KSGD_EXP_AUTO form without any host synchronisation.  The
 * exponent is left in *exp_theta_dev (device int32, 4-byte aligned) for whoever needs it on
 * the device (kahan_sgd_step_qgrad_dev reads gradient exponents from such an array).
 * scratch: device, at least 8 bytes, 4-byte aligned, zero on the first call (every call
 * leaves it zero again); calls that share a scratch must run one after the other.
 */
#define KSGD_EXP_AUTO INT32_MIN
int kahan_sgd_import(const float* src, void* theta, void* comp, int64_t numel, int32_t theta_bits,
                     int32_t comp_bits, int32_t overlap_k, int32_t exp_theta, int32_t* exp_theta_out,
                     void* scratch, void* cuda_stream);
int kahan_sgd_import_dev(const float* src, void* theta, void* comp, int64_t numel, int32_t theta_bits,
                         int32_t comp_bits, int32_t overlap_k, int32_t* exp_theta_dev, void* scratch,
                         void* cuda_stream);

/*
 * Dynamic fixed-point -> fp32: dst[i] = fl32(Q_theta*2^e + Q_c*2^(e-s)), the exact value of
 * theta + c rounded once.  dst: device, fp32[numel].  Enqueues only.
 */
int kahan_sgd_export(const void* theta, const void* comp, float* dst, int64_t numel, int32_t theta_bits,
                     int32_t comp_bits, int32_t overlap_k, int32_t exp_theta, void* cuda_stream);

/*
 * Bit-width of the last fully-connected layer in front of a softmax (Section 3, Eq. 5):
 * the smallest integer larger than log2(n_classes - 1) + log2(2 / alpha), 0 < alpha < 1
 * (the paper suggests alpha = 0.5).  Host-only.  Returns 0 for invalid arguments.
 */
int32_t kahan_sgd_classifier_bits(int64_t n_classes, double alpha);

/* Static text for a KSGD_* code. */
const char* kahan_sgd_strerror(int code);

/* Text of the last CUDA runtime error seen by the calling thread ("" if none). */
const char* kahan_sgd_last_cuda_error(void);

/* Number of this library's kernels launched by the calling process since load. */
uint64_t kahan_sgd_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* KAHAN_SGD_H_ */
