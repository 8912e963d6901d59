/* mp.h -- C ABI of the mixed-precision training step of a stack of linear layers,
 * for NVIDIA B200 (sm_100a) only.
 *
 * The operations are those of the paper "Mixed-Precision Training for NLP and Speech
 * Recognition with OpenSeq2Seq" (arXiv 1805.10387), Section 3:
 *   Section 3.1  matrix products with FP16 operands and FP32 accumulation; a loss scale S
 *                chosen from an inspection of the gradients and applied to the next step;
 *                an FP32 master copy of the weights;
 *   Section 3.2  FP16 gradients converted to FP32, optimizer run on the FP32 master,
 *                master converted back to the FP16 working copy;
 *   Section 3.3  weight decay formed from the FP32 master, not from the FP16 copy.
 *
 * Conventions
 *   - Every matrix is row-major.  FP16 means IEEE binary16 stored as 16-bit words.
 *   - Every tensor pointer is a DEVICE pointer owned by the caller and must be 16-byte
 *     aligned; leading dimensions (ld*) are in elements and multiples of 8.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All work is
 *     asynchronous on that stream; only mp_state_read* synchronise.
 *   - Every function returns an mp_status.  Nothing throws or aborts.  Argument errors are
 *     found on the host before anything is launched.  Numeric overflow is NOT an error: it
 *     is state (found_inf, skipped) held on the device.
 *   - FP32 -> FP16 conversions round to nearest even, overflow to +-inf (never saturate)
 *     and keep subnormals.
 *   - The library owns only mp_state and mp_update_plan objects.  It runs on the device
 *     that is current when a function is called; objects belong to the device they were
 *     created on.
 *   - Calls may come from several host threads.  The one-time set-up that a first call does per
 *     device and per kernel flavour (attribute, occupancy and symbol queries) is serialised
 *     inside the library; a state or plan object must not be used by two threads at once.
 *   - Device-side errors.  Every wait inside a kernel is bounded.  A product kernel whose wait
 *     runs out stops taking work, releases what it holds and returns; it records
 *     MP_ERR_TIMEOUT in a device-wide status word and, when the call was given a state, in
 *     state->status.  While either is set, mp_master_update writes nothing and
 *     mp_loss_scale_update changes nothing (it copies the device-wide word into
 *     state->status): the training state is frozen as it was before the faulty step.  The host
 *     learns of it from mp_state_read (status) or mp_gemm_device_status, and resumes with
 *     mp_gemm_device_status (which clears the device-wide word) followed by mp_state_write
 *     with status = 0.
 */
#ifndef MP_H_
#define MP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MP_OK = 0,
  MP_ERR_INVALID_ARG = -1,      /* null pointer, non-positive size, ld < extent, bad enum  */
  MP_ERR_ALIGNMENT = -2,        /* pointer not 16-byte aligned or ld not a multiple of 8   */
  MP_ERR_UNSUPPORTED_ARCH = -3, /* current device is not compute capability 10.x           */
  MP_ERR_CUDA = -4,             /* a CUDA runtime/driver call failed; see mp_last_error    */
  MP_ERR_TIMEOUT = -5,          /* a bounded device-side wait expired (reported in status) */
  MP_ERR_NOMEM = -6,            /* allocation failed or workspace too small                */
  MP_ERR_TOO_LARGE = -7         /* size beyond a stated maximum                            */
} mp_status;

typedef struct mp_state mp_state;             /* device-resident scaler + flag + log        */
typedef struct mp_update_plan mp_update_plan; /* device table over the tensors of an update */

/* Loss-scale policy (Section 3.1, item 1).  dynamic != 0: halve S (not below min_scale) after
 * a step whose gradients held an inf/NaN, double it (not above max_scale) after
 * growth_interval clean steps in a row.  dynamic == 0: S stays init_scale (static loss
 * scaling); an overflow step is still skipped.
 * overflow_tolerance = H > 1 selects a second policy that the paper does not describe: S is
 * halved at the H-th overflow since S last changed (a doubling clears the count too), so an
 * isolated overflow costs a skipped step but no halving.  Every overflow step is still
 * skipped and still restarts the run of clean steps.  H = 1 is the plain rule. */
typedef struct {
  float init_scale;        /* > 0 */
  float min_scale;         /* > 0 */
  float max_scale;         /* >= min_scale */
  int32_t growth_interval; /* >= 1 */
  int32_t dynamic;
  int32_t overflow_tolerance; /* >= 1 */
} mp_scaler_config;

typedef enum { MP_OPT_ADAM = 0, MP_OPT_MOMENTUM = 1 } mp_opt_kind;

/* Optimizer run on the FP32 master (Section 3.2).  Adam: m = b1 m + (1-b1) g,
 * v = b2 v + (1-b2) g^2, w -= lr (m/(1-b1^t)) / (sqrt(v/(1-b2^t)) + eps), t = number of
 * applied steps including this one.  Momentum: u = mu u + g, w -= lr u.
 * weight_decay adds weight_decay * w32 to g before the moments (Section 3.3). */
typedef struct {
  int32_t kind; /* mp_opt_kind */
  float lr, beta1, beta2, eps, momentum, weight_decay;
} mp_optim_config;

/* Host copy of the device state, filled by mp_state_read. */
typedef struct {
  float scale;         /* S that the NEXT step will use                                     */
  float min_scale, max_scale;
  int32_t growth_interval, dynamic;
  int32_t good_steps;  /* clean steps since S last changed                                  */
  int32_t found_inf;   /* flag accumulated by the current step so far                       */
  int32_t status;      /* MP_OK or the first device-side error (MP_ERR_TIMEOUT), see above  */
  int32_t overflow_tolerance;
  int32_t strikes;     /* overflows since S last changed (dynamic scale with tolerance 1:
                          always 0; static scale: S never changes, so every overflow counts) */
  int64_t t;           /* applied optimizer steps                                           */
  int64_t step;        /* all steps                                                         */
  int64_t skipped;     /* overflow steps                                                    */
} mp_state_host;

/* One record per mp_loss_scale_update call, kept in a device ring of MP_LOG_CAPACITY. */
typedef struct {
  int64_t step;
  int64_t t;           /* after the step */
  float scale_before, scale_after;
  int32_t found_inf, good_steps;
} mp_log_record;
#define MP_LOG_CAPACITY 4096

/* ---- the five calls of the step ------------------------------------------------------ */

/* Forward product (Section 3.1): Y[M,N] = rn16( sum_k X[m,k] * W[k,n] ), FP32 accumulation.
 * X16 [M,K] ldx>=K, W16 [K,N] ldw>=N, Y16 [M,N] ldy>=N, all FP16 device buffers.
 * workspace: device scratch of at least mp_gemm_workspace_bytes(M,K,N,MP_OP_FWD) bytes
 * (may be NULL when that is 0).  Errors: INVALID_ARG, ALIGNMENT, NOMEM (workspace too
 * small), UNSUPPORTED_ARCH, CUDA. */
int mp_linear_fwd(const void* X16, int64_t ldx, const void* W16, int64_t ldw, void* Y16,
                  int64_t ldy, int64_t M, int64_t K, int64_t N, void* workspace,
                  size_t workspace_bytes, void* stream);

/* Data gradient (Section 3.2, "gradients are in FP16"): dX[M,K] = rn16( sum_n dY[m,n] *
 * W[k,n] ).  W is read in place as stored (no transposed copy). */
int mp_linear_bwd_dgrad(const void* dY16, int64_t lddy, const void* W16, int64_t ldw,
                        void* dX16, int64_t lddx, int64_t M, int64_t K, int64_t N,
                        void* workspace, size_t workspace_bytes, void* stream);

/* Weight gradient: dW[K,N] = rn16( sum_m X[m,k] * dY[m,n] ), still multiplied by S.
 * If state != NULL, state->found_inf is set when any element written to dW16 is inf or NaN
 * (the gradient inspection of Section 3.1, item 1, done where the gradient is produced). */
int mp_linear_bwd_wgrad(const void* X16, int64_t ldx, const void* dY16, int64_t lddy,
                        void* dW16, int64_t lddw, int64_t M, int64_t K, int64_t N,
                        mp_state* state, void* workspace, size_t workspace_bytes, void* stream);

/* Fused master update over every tensor of the plan (Section 3.2): if the step's flag is
 * clear, g = float(g16) * (1/S), optimizer on w32 (and m, v), w16 = rn16(w32); if it is set,
 * nothing is written.  check_mode 0: trust state->found_inf as set by the wgrad calls;
 * check_mode 1: first inspect every g16 of the plan (sets state->found_inf), then update.
 * S, t and the flag are read on the device; nothing returns to the host. */
int mp_master_update(mp_update_plan* plan, mp_state* state, const mp_optim_config* opt,
                     int check_mode, void* stream);

/* Loss-scale state machine (Section 3.1, item 1: the scale for the next step is chosen from
 * this step's inspection).  Flag set: S = max(S/2, min_scale), good = 0, skipped++.
 * Flag clear: t++, good++, and when good == growth_interval: S = min(2S, max_scale), good = 0.
 * Then the flag is cleared, step++ and a log record is appended.  One tiny kernel. */
int mp_loss_scale_update(mp_state* state, void* stream);

/* Weight gradient for callers that must not allocate.  (The paper has no counterpart: this is
 * a packaging variant of mp_linear_bwd_wgrad, same arithmetic, same results bit for bit.)
 *
 * Who needs it: code that runs where device allocation is off the table -- a training or
 * serving runtime that has already handed all free device memory to its own pool, so that a
 * cudaMalloc would fail; a step that must not hit the implicit device-wide synchronisation an
 * allocation or free causes; a plugin whose host forbids allocator calls inside its callbacks.
 * Such callers also may have no spare buffer to lend as `workspace`.
 *
 * Differences from mp_linear_bwd_wgrad: there is no workspace argument.  The split-reduction
 * scratch is an array built into the library image, MP_STATIC_SCRATCH_BYTES (32 MiB) per GPU,
 * reserved on every GPU that loads the library until the process exits.  Sizes whose scratch
 * need (mp_gemm_workspace_bytes(M,K,N,MP_OP_WGRAD)) exceeds it are refused with
 * MP_ERR_TOO_LARGE and nothing is launched.  The call makes no cudaMalloc/cudaFree and uses no
 * allocating library routine.
 *
 * The first call on each device looks up the array's device address (one cheap runtime query,
 * no allocation, done with that device current), and like every product call the first one per
 * device and kernel flavour also sets kernel attributes and asks for occupancy; make a first
 * call with sizes of the same class (K above or at most 128, i.e. the same kernel flavour)
 * before starting any stream capture.  All calls on a device share the one array: two calls whose kernels may
 * overlap on the GPU (different streams) race on it and must be ordered by the caller.  The
 * array keeps whatever the previous call left; that is harmless because each call overwrites
 * every partial sum it later reads, so nothing has to start at zero. */
#define MP_STATIC_SCRATCH_BYTES (32u << 20)
int mp_linear_bwd_wgrad_static(const void* X16, int64_t ldx, const void* dY16, int64_t lddy,
                               void* dW16, int64_t lddw, int64_t M, int64_t K, int64_t N,
                               mp_state* state, void* stream);
/* Size of that built-in scratch in bytes (equals MP_STATIC_SCRATCH_BYTES). */
size_t mp_static_scratch_bytes(void);

/* ---- several independent layers of one shape in one launch ------------------------------
 * The products of Section 3.1 for `count` (1 .. mp_max_group()) layers that have the same M, K,
 * N and leading dimensions and do not depend on one another (the query, key and value
 * projections of an attention block; the per-layer gate products of a stack whose layers are
 * fed independently).  X16, W16, Y16 ... are host arrays of `count` device pointers; each
 * problem obeys the rules of the single call of the same name and gets that call's result (bit
 * for bit when both split the reduction the same way; otherwise the FP32 partial sums are added
 * in another, equally fixed order).  One launch walks the tiles of all problems, so a product too small to fill
 * the GPU's waves on its own does not leave SMs idle.  workspace: at least
 * mp_gemm_workspace_bytes_grouped(count, M, K, N, op) bytes.  Errors as for the single calls;
 * INVALID_ARG also for count outside 1 .. mp_max_group(). */
int mp_linear_fwd_grouped(int count, const void* const* X16, int64_t ldx, const void* const* W16,
                          int64_t ldw, void* const* Y16, int64_t ldy, int64_t M, int64_t K, int64_t N,
                          void* workspace, size_t workspace_bytes, void* stream);
int mp_linear_bwd_dgrad_grouped(int count, const void* const* dY16, int64_t lddy, const void* const* W16,
                                int64_t ldw, void* const* dX16, int64_t lddx, int64_t M, int64_t K,
                                int64_t N, void* workspace, size_t workspace_bytes, void* stream);
/* ORs "an inf or NaN was stored" of every problem into state->found_inf (state may be NULL). */
int mp_linear_bwd_wgrad_grouped(int count, const void* const* X16, int64_t ldx, const void* const* dY16,
                                int64_t lddy, void* const* dW16, int64_t lddw, int64_t M, int64_t K,
                                int64_t N, mp_state* state, void* workspace, size_t workspace_bytes,
                                void* stream);
/* The grouped forward product with the bias and activation of mp_linear_fwd_act: bias16 is a
 * host array of `count` device pointers (or NULL for no bias), one activation for all. */
int mp_linear_fwd_act_grouped(int count, const void* const* X16, int64_t ldx, const void* const* W16,
                              int64_t ldw, const void* const* bias16, void* const* Y16, int64_t ldy,
                              int64_t M, int64_t K, int64_t N, int act, float clip, void* workspace,
                              size_t workspace_bytes, void* stream);
/* Largest `count` the grouped calls take. */
int mp_max_group(void);

/* ---- layers with a bias and an activation ------------------------------------------------
 * The models of the paper's Section 5 follow their dense products with a bias and a
 * nonlinearity (ReLU in the Transformer feed-forward block, clipped ReLU in DeepSpeech2).  The
 * paper gives no arithmetic for them; this library's reading: the FP16 bias is added to the
 * FP32 sum before the single rounding to FP16, the activation acts on that FP32 value, and the
 * backward pass zeroes the FP16 data gradient where the stored FP16 output of the activated
 * layer is outside the activation's linear range. */
typedef enum { MP_ACT_NONE = 0, MP_ACT_RELU = 1, MP_ACT_CLIPPED_RELU = 2 } mp_activation;

/* Y[M,N] = rn16( act( sum_k X[m,k] W[k,n] + bias[n] ) ).  bias16: N FP16 values, 16-byte aligned,
 * or NULL.  act: mp_activation; clip: upper bound of MP_ACT_CLIPPED_RELU (min(max(x,0),clip)).
 * Other arguments and errors as mp_linear_fwd. */
int mp_linear_fwd_act(const void* X16, int64_t ldx, const void* W16, int64_t ldw, const void* bias16,
                      void* Y16, int64_t ldy, int64_t M, int64_t K, int64_t N, int act, float clip,
                      void* workspace, size_t workspace_bytes, void* stream);

/* dX[m,k] = rn16( sum_n dY[m,n] W[k,n] ) where A[m,k] passes the activation (A > 0 for ReLU,
 * 0 < A < clip for clipped ReLU), else +0.  A16 [M,K] (lda >= K) is this layer's input, i.e.
 * the activated FP16 output of the layer below; it may alias nothing that is written.  With
 * MP_ACT_NONE the call equals mp_linear_bwd_dgrad and A16 may be NULL. */
int mp_linear_bwd_dgrad_act(const void* dY16, int64_t lddy, const void* W16, int64_t ldw,
                            const void* A16, int64_t lda, void* dX16, int64_t lddx, int64_t M,
                            int64_t K, int64_t N, int act, float clip, void* workspace,
                            size_t workspace_bytes, void* stream);

/* db[n] = rn16( sum_m dY[m,n] ), FP32 accumulation in a fixed order (results do not depend on
 * timing), still multiplied by S.  Sets state->found_inf if a stored value is inf or NaN (state
 * may be NULL).  workspace: at least mp_bias_grad_workspace_bytes(M,N) bytes of device scratch. */
int mp_bias_grad(const void* dY16, int64_t lddy, void* db16, int64_t M, int64_t N, mp_state* state,
                 void* workspace, size_t workspace_bytes, void* stream);
size_t mp_bias_grad_workspace_bytes(int64_t M, int64_t N);
/* The same for `count` (1 .. mp_max_group()) gradients of one shape and row pitch in one pair of launches: dY16 and
 * db16 are host arrays of `count` device pointers; every result is the single call's, bit for bit.
 * workspace: at least count * mp_bias_grad_workspace_bytes(M,N) bytes. */
int mp_bias_grad_grouped(int count, const void* const* dY16, int64_t lddy, void* const* db16, int64_t M,
                         int64_t N, mp_state* state, void* workspace, size_t workspace_bytes, void* stream);

/* LSTM cell for a gate product G = [x;h] W of 4H columns in the order i, f, g, o (the GNMT-like
 * layers of Section 5; the paper gives no arithmetic, so: FP16 gates and states in memory, the
 * cell evaluated in FP32 with sigma(x) = 1/(1+exp(-x)) and tanh, one rounding per output).
 *   c_new = sigma(f) c_prev + sigma(i) tanh(g),   h = sigma(o) tanh(c_new)
 * G16 [M,4H] with ldg >= 4H; c_prev16, c_new16, h16 dense [M,H]; H and ldg multiples of 8. */
int mp_lstm_cell_fwd(const void* G16, int64_t ldg, const void* c_prev16, void* c_new16, void* h16,
                     int64_t M, int64_t H, void* stream);

/* Backward of the cell from the stored FP16 gates and states: dh16 is the gradient at h,
 * dc_in16 the gradient arriving at c_new from the next time step (NULL = none).  Writes dG16
 * [M,4H] (gradient at the gate pre-activations, the dY of the gate product's backward calls)
 * and dc_prev16 [M,H]; tanh(c_new) is taken from the stored FP16 c_new.  Gradients stay
 * multiplied by the loss scale. */
int mp_lstm_cell_bwd(const void* G16, int64_t ldg, const void* c_prev16, const void* c_new16,
                     const void* dh16, const void* dc_in16, void* dG16, int64_t lddg, void* dc_prev16,
                     int64_t M, int64_t H, void* stream);

/* ---- auxiliaries --------------------------------------------------------------------- */

enum { MP_OP_FWD = 0, MP_OP_DGRAD = 1, MP_OP_WGRAD = 2 };

/* Scratch bytes the GEMM of `op` needs for these sizes (0 when it needs none). */
size_t mp_gemm_workspace_bytes(int64_t M, int64_t K, int64_t N, int op);
/* The same for a grouped call over `count` problems (0 for a count the calls refuse). */
size_t mp_gemm_workspace_bytes_grouped(int count, int64_t M, int64_t K, int64_t N, int op);

/* dY16[i] = rn16( S * g32[i] ), S read from the device state (Section 3.1, item 1: the loss
 * is scaled; for a linear stack that is the gradient entering the top layer). */
int mp_scale_upstream(const float* g32, void* dY16, int64_t n, const mp_state* state,
                      void* stream);

/* Sets state->found_inf if any of the n FP16 values at g16 is inf or NaN. */
int mp_check_finite(const void* g16, int64_t n, mp_state* state, void* stream);

int mp_state_create(const mp_scaler_config* cfg, mp_state** out);
int mp_state_destroy(mp_state* state); /* NULL is accepted */
/* Synchronises `stream`, then copies the device state to *out. */
int mp_state_read(mp_state* state, mp_state_host* out, void* stream);
/* Overwrites the device state (resume from a checkpoint); synchronises `stream`. */
int mp_state_write(mp_state* state, const mp_state_host* in, void* stream);
/* Copies up to max_records of the most recent log records, oldest first, to out (host);
 * *n_out receives the count.  Synchronises `stream`. */
int mp_state_read_log(mp_state* state, mp_log_record* out, int max_records, int* n_out,
                      void* stream);

/* Data-parallel runs whose ranks each inspect only a slice of the summed gradients (Section 4
 * of the paper: replicas that exchange gradients; the sharded-update schedule) agree on the
 * overflow flag by reducing one word across ranks.  These two calls move the flag between the
 * device state and a caller-owned int32 device word, asynchronously on `stream`, with no host
 * round trip: export writes *word = (found_inf != 0); import ORs (*word != 0) into found_inf.
 * word: device pointer, 4-byte aligned. */
int mp_state_export_flag(const mp_state* state, int32_t* word, void* stream);
int mp_state_import_flag(mp_state* state, const int32_t* word, void* stream);

/* Plan over n tensors: g16[i], w16[i] FP16 and w32[i], m[i], v[i] FP32 device buffers of
 * count[i] elements each (count[i] == 0 is legal and skipped).  v may be NULL for a plan
 * used only with momentum (m then holds the momentum buffer).  The pointer arrays are host
 * arrays and are copied; the tensors stay the caller's. */
int mp_update_plan_create(int n, void* const* g16, void* const* w32, void* const* m,
                          void* const* v, void* const* w16, const int64_t* count,
                          mp_update_plan** out);
int mp_update_plan_destroy(mp_update_plan* plan); /* NULL is accepted */

/* Error-path self-test (not one of the step's calls; the paper has no counterpart).  Launches
 * the forward product's kernel on ONE output tile (M <= 128, N <= 256; arguments otherwise as
 * mp_linear_fwd) with its loader told to fetch nothing and every pipeline wait limited to
 * wait_us microseconds (1 .. 2000000).  No copy is ever in flight: the waits run out, the
 * kernel records MP_ERR_TIMEOUT (device-wide and, if state != NULL, in state->status), frees
 * its tensor memory and returns without writing Y16.  It exists so that the library's
 * reaction to an expired wait can be exercised on a healthy GPU. */
int mp_selftest_wait_timeout(const void* X16, int64_t ldx, const void* W16, int64_t ldw, void* Y16,
                             int64_t ldy, int64_t M, int64_t K, int64_t N, int64_t wait_us,
                             mp_state* state, void* stream);

/* Synchronises the device and reports in *out the first device-side error recorded by a GEMM
 * kernel since the last call (MP_OK, or MP_ERR_TIMEOUT when a bounded wait on a pipeline
 * barrier expired; the kernel then skipped its remaining work and returned).  Clears it. */
int mp_gemm_device_status(int* out);

/* Message of the last error on the calling thread ("" if none). */
const char* mp_last_error(void);

/* Number of kernels this library has launched in the calling process (for accounting). */
int64_t mp_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* MP_H_ */
