/*
 * dq.h -- C ABI of libdq: one round of double quantization on one NVIDIA B200 (sm_100a).
 *
 * Method: "Double Quantization for Communication-Efficient Distributed Optimization"
 * (AsyLPG = Algorithm 1, Sparse-AsyLPG = Algorithm 2, Acc-AsyLPG = Algorithm 3).  The problem is
 * eq. (1): min_{x in Omega} f(x) + h(x), f = (1/n) sum_i f_i.  Here f_i is the logistic loss
 * log(1 + exp(-y_i <a_i, x>)) with labels y_i = +-1, h = lambda1 |x|_1 + (lambda2/2) |x|^2, and Omega is
 * the box [box_lo, box_hi]^d.  M workers are simulated as independent lanes of one GPU; a "round" is one
 * inner iteration (Algorithm 1 steps 6-13) in which all M workers answer the same broadcast model and the
 * master averages their messages before one prox step.
 *
 * General rules
 *   - Every function returns a DQ_* status and never throws, exits or allocates behind the caller's back
 *     except dq_create (which allocates the context's scratch) and dq_destroy (which frees it).
 *   - Unless a parameter is marked HOST, pointers are DEVICE pointers owned by the caller; they must stay
 *     valid until the stream work that uses them has finished.  Vectors are contiguous fp32.
 *   - Work is enqueued on the CUDA stream passed as `stream` (a cudaStream_t cast to void*; NULL is the
 *     default stream).  No call synchronises the device unless it says so.
 *   - Errors found on the host (bad argument, bad bit width, misaligned buffer) are returned immediately.
 *     Errors found by a kernel (non-finite norm, sparse message over capacity) set a sticky status word that
 *     dq_poll_status reads.  A vector that holds a NaN or an Inf is quantised to scale 0 and all-zero codes.
 *   - The gradient width b must be 2, 4 or 8; the model width b_x may be any of 2..11, the widths of Table 1
 *     (b = 1 would give 2^(b-1)-1 = 0 levels).  Up to 8 bits the rounding position keeps 15 fractional bits, then
 *     14, 13 and 12 for 9, 10 and 11 bits.
 *   - All random draws come from Philox4x32-10 with key = seed and counter
 *     (coordinate >> 3, round, worker, stream); the master's worker id is 0xFFFFFFFF; streams are
 *     0 model rounding, 1 gradient rounding, 2 sparsification mask, 3 minibatch sampling.  Equal
 *     (seed, round, inputs) give equal bytes from every stage of a round on the same kernel path: dense rows are
 *     summed in slot order, CSR rows on an exact integer grid, norms as integer maxima / integer sums.  (The
 *     one-cluster kernel and the separate kernels form a row's margin in different orders; each agrees with itself.)
 *     The exception is dq_epoch_begin: the epoch's full gradient is summed with double-precision atomics, so a
 *     coordinate of g_full may differ in its last place between two runs.
 *
 * Packed code layout (message of Section 3.1: 32 bits for delta plus b bits per coordinate): codes are b-bit
 * two's complement fields laid end to end: coordinate j occupies bits [j b, (j+1) b) of the message, bit k of the
 * message being bit k mod 8 of byte k / 8 (for b dividing 8: byte j / (8/b) at bit offset (j mod (8/b)) * b).  The
 * bytes of one message are padded with zeros to dq_packed_bytes(d, b), a multiple of 16.  delta is kept in a
 * separate fp32 array.
 */
#ifndef DQ_H_
#define DQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    DQ_OK = 0,
    DQ_ERR_ARG = 1,        /* NULL pointer, non-positive size, misaligned buffer                     */
    DQ_ERR_SHAPE = 2,      /* sizes inconsistent with the context (d, M, stride, capacity)            */
    DQ_ERR_BITS = 3,       /* b not in {2, 4, 8} or b_x outside 2..11                                 */
    DQ_ERR_NONFINITE = 4,  /* a vector to be quantised holds NaN or Inf                               */
    DQ_ERR_CAPACITY = 5,   /* a sparse message had more survivors than the buffers can hold           */
    DQ_ERR_CUDA = 6,       /* a CUDA runtime call failed                                              */
    DQ_ERR_TIMEOUT = 7     /* reserved                                                                */
};

enum { DQ_DENSE_F32 = 0, DQ_CSR_F32 = 1, DQ_DENSE_BF16 = 2 };   /* dq_data.format */
enum { DQ_MSG_DENSE = 0, DQ_MSG_SPARSE = 1 };                   /* dq_config.msg_format */
enum { DQ_MODEL_LOGISTIC = 0, DQ_MODEL_MLP = 1 };               /* dq_config.model */

/* The training set {a_i, y_i} of eq. (1).  values: DENSE_F32 [n][d] float; DENSE_BF16 [n][d] bfloat16;
 * CSR_F32 [nnz] float with col_idx [nnz] (ascending inside a row, < d) and row_ptr [n+1].  labels [n] = +-1.
 * All device pointers, read-only, 16-byte aligned. */
typedef struct {
    int32_t format; int32_t reserved;
    int64_t n, d;
    const void* values;
    const int32_t* col_idx;
    const int64_t* row_ptr;
    const float* labels;
} dq_data;

/* Inputs of Algorithms 1-3 that stay fixed during a run. */
typedef struct {
    int64_t d;                 /* model size                                                            */
    int32_t M, B;              /* simulated workers; minibatch rows per worker and round                */
    int32_t bx, b;             /* bits for the model (step 8) and for the gradient (step 12)            */
    float lambda1, lambda2;    /* h = lambda1 |x|_1 + (lambda2/2) |x|^2                                  */
    float box_lo, box_hi;      /* Omega = [box_lo, box_hi]^d; -INFINITY/+INFINITY for no constraint      */
    int32_t sparsify;          /* 1: Algorithm 2 (eq. (4) before quantising)                            */
    float phi;                 /* sparsity budget sum p_i; <= 0 or too large: |alpha|_1/|alpha|_inf (Lemma 2) */
    int32_t msg_format;        /* DQ_MSG_SPARSE needs sparsify = 1                                      */
    int32_t accelerated;       /* 1: Algorithm 3                                                        */
    int32_t snapshot_flag;     /* 1: send one flag bit instead of the model when x equals the snapshot  */
    int32_t no_graph;          /* 1: dq_round launches its kernels one by one instead of replaying a CUDA graph */
    uint64_t seed;
    int64_t sparse_cap;        /* entries per worker in the context's own sparse message buffers; 0: d   */
    float mu;                  /* > 0: dq_round picks b_x in 2..11 each round by condition (3)/(6); 0: fixed bx */
    int32_t sequential;        /* 1: master applies the M messages one by one, one prox step each (Algorithm 1 step 9 as
                                  written; message w is w steps stale, delay <= M-1); 0: one step on their average */
    int32_t model;             /* DQ_MODEL_LOGISTIC (default) or DQ_MODEL_MLP: the 3-layer fully connected network of
                                  Section 5.2, in -> hidden (ReLU) -> classes with softmax cross-entropy.  For the network
                                  the data must be DQ_DENSE_F32 with labels = class index, data.d = number of inputs, and
                                  d = hidden*(in+1) + classes*(hidden+1) with x = [W1 (hidden x in), b1, W2 (classes x hidden), b2] */
    int32_t hidden, classes;      /* hidden + 3*classes <= 3072 */
    int32_t no_fused;          /* 0: merged kernels where they apply (the one-cluster round, quantiser + master in one kernel, the
                                  one-pass dense gradient carrying the whole round); 1: every stage as its own kernel(s), the plan
                                  the merged ones are tested against; 2: like 1, but the dense gradient stage stays one pass */
    int32_t max_delay;         /* tau of Assumption 3: dq_round keeps the last tau + 1 broadcast models of the epoch so that
                                  workers can be made to lag (dq_set_delays); 0: every worker uses the current broadcast */
    int32_t tensor_cores;      /* 1: the one-pass dense gradient forms X (xhat - xsnap) and X^T r of bfloat16 rows (d a multiple of
                                  16) as bf16 tensor-core MMAs with fp32 accumulation, the fp32 factors split into three bfloat16
                                  terms; 0: fp32 FMAs on CUDA cores (the default: measured faster, see the profiles) */
    int32_t delay_across_epochs; /* with max_delay > 0: 1 lets a delay reach back into the previous epoch (the worker then evaluates
                                  the previous epoch's low-precision model against the new snapshot and full gradient); 0 (default)
                                  cuts a delay to the rounds the epoch has had.  Such a context launches its rounds kernel by
                                  kernel (no captured graph) */
} dq_config;

/* Optimiser state, all [d] fp32 device vectors owned by the caller.  y and x_sum are used by Algorithm 3
 * only (may be NULL otherwise).  norm_x is one device float holding ||x||_inf, maintained by the library.
 * z_snap [n] caches the margins <a_i, x_snap> (written at epoch begin). */
typedef struct {
    float* x; float* x_snap; float* g_full; float* y; float* x_sum;
    float* norm_x; float* z_snap;
} dq_state;

/* M worker messages.  Dense: codes [M][stride] bytes (stride >= dq_packed_bytes(d, b), multiple of 16) and
 * scale [M] (= delta).  Sparse (Section 4.2's encoding: position then value per nonzero of beta): nnz [M],
 * idx [M][cap] ascending coordinate indices, and the value codes packed b bits each in list order in
 * codes [M][stride] (stride >= dq_packed_bytes(cap, b)). */
typedef struct {
    uint8_t* codes; int64_t stride; float* scale;
    uint32_t* idx; int64_t cap; uint32_t* nnz;
} dq_msgs;

typedef struct dq_ctx dq_ctx;

/* Bytes of one packed message of `count` codes of b bits, padded to a multiple of 16. */
int64_t dq_packed_bytes(int64_t count, int b);

/* Create a context for `cfg` on the current device.  `data` may be NULL when only the codec entry points
 * (dq_quantize_model, dq_quantize_sparsify_pack, dq_master_unpack_aggregate_prox, dq_codec_round,
 * dq_unpack) will be used.  Allocates the context's scratch (norms, message buffers for dq_round,
 * survivor staging); the structs are copied, the arrays they point to are not. */
int dq_create(dq_ctx** out, const dq_config* cfg, const dq_data* data);
int dq_destroy(dq_ctx* ctx);

/* Epoch boundary (Algorithm 1 steps 3-5 and 14; Algorithm 3 steps 3-5 and 15).
 * Algorithms 1/2: x_snap <- x.  Algorithm 3: if rounds have run since the last call, x_snap <- x_sum / m
 * (m = number of those rounds) and x_sum <- 0; y is carried over; x <- x_snap + theta (y - x_snap).
 * Then g_full <- grad f(x_snap) in full precision over all n rows, z_snap <- margins, norm_x <- ||x||_inf. */
int dq_epoch_begin(dq_ctx* ctx, dq_state* st, float theta, void* stream);

/* Master step 8: delta_x = ||x||_inf / (2^(bx-1)-1); codes_x <- packed Q_(delta_x,bx)(x) (Section 3.1).
 * norm_x: device float holding ||x||_inf, or NULL to have it computed.  codes_x must hold
 * dq_packed_bytes(d, bx) bytes; delta_x is one device float. */
int dq_quantize_model(dq_ctx* ctx, const float* x, const float* norm_x, uint32_t round,
                      uint8_t* codes_x, float* delta_x, void* stream);

/* Model precision (condition (3); condition (6) for Algorithm 3 passes theta_s * mu): writes to *bits (device int)
 * the smallest width b in 2..11 (the widths of Table 1) with  E_Q ||Q_(delta,b)(x) - x||^2 <= mu ||x - x_snap||^2,
 * 11 if none, where the left side is the closed form sum_i (x_i - z_i)(z_i + delta - x_i) of rule (i).  stats
 * (device double[11], may be NULL) receives the expected errors at 2..11 bits and ||x - x_snap||^2.  norm_x: device
 * ||x||_inf or NULL. */
int dq_select_model_bits(dq_ctx* ctx, const float* x, const float* x_snap, const float* norm_x, float mu,
                         int32_t* bits, double* stats, void* stream);

/* Width chosen by the last dq_round of a context with mu > 0 (synchronises `stream`); 0 after a snapshot round. */
int dq_last_model_bits(dq_ctx* ctx, int32_t* bits_host, void* stream);

/* Worker step 11 for all M workers: alpha_w = (1/B) sum_{a in batch_w} [grad f_a(xhat) - grad f_a(x_snap)],
 * xhat = dequantised broadcast model (code * delta_x), or x_snap itself when is_snapshot != 0 (flag bit of
 * the "Model Parameter Quantization" paragraph; codes_x/delta_x are then ignored).  batch_idx: [M][B] row
 * indices (int32) or NULL to draw them from the batch stream (worker w samples its own contiguous
 * partition of the rows, with replacement).  Outputs alpha [M][d], norm_inf [M] = ||alpha_w||_inf. */
int dq_worker_grad(dq_ctx* ctx, const uint8_t* codes_x, const float* delta_x, int is_snapshot,
                   const dq_state* st, uint32_t round, const int32_t* batch_idx,
                   float* alpha, float* norm_inf, void* stream);

/* ||v_w||_inf for the M rows of v [M][d] into norm_inf [M] (device floats): the numerator of the scale
 * delta of Algorithm 1 steps 8 and 12, for callers whose gradient producer does not supply it. */
int dq_norm_inf(dq_ctx* ctx, const float* v, int M, float* norm_inf, void* stream);

/* Worker steps 12(-13) for all M workers: optional sparsification by eq. (4) with Lemma 2's probabilities,
 * then delta = ||.||_inf / (2^(b-1)-1), Q_(delta,b), and bit packing into `out`.
 * v [M][d]; norm_inf [M] = ||v_w||_inf exactly as produced by dq_worker_grad or dq_norm_inf, or NULL to have it
 * computed.  A value below the true maximum gives unspecified codes for the coordinates that exceed it. */
int dq_quantize_sparsify_pack(dq_ctx* ctx, const float* v, const float* norm_inf, uint32_t round,
                              dq_msgs* out, void* stream);

/* Master step 9: g = (1/M) sum_w dequantised message w; u = g + g_full;
 * Algorithms 1/2: x <- prox_{eta h}(x - eta u).
 * Algorithm 3:    y <- prox_{eta h}(y - eta u); x <- x_snap + theta (y - x_snap); x_sum <- x_sum + x.
 * Also writes ||x||_inf of the new model to st->norm_x. */
int dq_master_unpack_aggregate_prox(dq_ctx* ctx, const dq_msgs* msgs, dq_state* st, float eta, float theta,
                                    void* stream);

/* One whole round on the context's own message buffers: model quantisation, M worker gradients,
 * (sparsify,) quantise, pack, master step, bit accounting.  bits_down / bits_up (device uint64, may be
 * NULL) receive the transmitted bits of this round by the paper's message sizes: down = M (32 + bx d), or M
 * flag bits on a snapshot round; up = sum_w (32 + b d) dense, sum_w (32 + nnz_w (ceil(log2 d) + b)) sparse.
 * The round is a snapshot round when snapshot_flag is set and it is the first round after dq_epoch_begin
 * (Algorithm 3: of the first epoch only).
 * Unless no_graph is set, the first non-snapshot round on a given set of state/counter pointers records its
 * kernel sequence as a CUDA graph (this allocates); later rounds replay it.  The graph's kernels read (round,
 * eta, theta) from device memory, where the round's last kernel advances the round number, so consecutive rounds
 * with the same step sizes cost one graph launch; anything else costs one small kernel that sets the three values.
 * Calling with other pointers records again.
 * Small problems (logistic model on DENSE_F32 or CSR_F32 data, dense messages, synchronous master, fixed b_x,
 * d <= 8192, M <= 16, B <= 1024) skip the graph unless no_fused is set: their non-snapshot rounds run in ONE
 * kernel on one thread-block cluster (block w is worker w; the blocks meet at the cluster barrier around the
 * master step), because
 * separate kernels would spend their time in launch gaps.  Results, buffers and layouts are the same. */
int dq_round(dq_ctx* ctx, dq_state* st, uint32_t round, float eta, float theta,
             uint64_t* bits_down, uint64_t* bits_up, void* stream);

/* Delays (Algorithm 1 step 11 evaluates the gradient at x_{D(t)}; Assumption 3: t - D(t) <= tau).  delays (HOST,
 * [M], each in 0..max_delay; NULL: all zero) says for every worker how many rounds before the current one the model
 * it works on was broadcast; it holds for the following dq_round calls until set again.  A delay is cut to the
 * number of rounds the epoch has had (the first round's workers all see the current model), or, with
 * cfg.delay_across_epochs, to the rounds the context has had since its first epoch began.  Needs
 * cfg.max_delay > 0; both models take delays (for the network the kept broadcasts are the low-precision parameters
 * themselves).  Such a context replays its rounds as a captured graph like any other (the kernels pick the
 * broadcast of a lagging worker from a round counter kept on the device), but not in the one-cluster kernel.
 * Copies synchronously. */
int dq_set_delays(dq_ctx* ctx, const int32_t* delays);

/* nrounds consecutive rounds round0, round0 + 1, ... of the same epoch with the same (eta, theta), as by
 * dq_round called once per round (Algorithm 1 steps 6-13 repeated; the caller places dq_epoch_begin between
 * epochs).  Where the one-cluster kernel applies, all non-snapshot rounds of the call run in a single launch;
 * otherwise the rounds are enqueued one after the other.  bits_down / bits_up hold the last round's counts. */
int dq_rounds(dq_ctx* ctx, dq_state* st, uint32_t round0, int32_t nrounds, float eta, float theta,
              uint64_t* bits_down, uint64_t* bits_up, void* stream);

/* The round without its gradient stage, for callers that bring their own M gradient vectors v [M][d]:
 * quantise(+sparsify)+pack into the context's buffers, master step on `st`, then model quantisation of the
 * new x into codes_x / delta_x. */
int dq_codec_round(dq_ctx* ctx, const float* v, dq_state* st, uint32_t round, float eta, float theta,
                   uint8_t* codes_x, float* delta_x, void* stream);

/* Same as dq_codec_round with HOST buffers: copies v [M][d] to the device, runs the round on the context's
 * device-resident state (set by dq_codec_host_setup), copies codes_x (dq_packed_bytes(d, bx) bytes) and
 * delta_x back, and synchronises the stream.  Host buffers should be pinned for full copy speed. */
int dq_codec_host_setup(dq_ctx* ctx, const float* x_host, const float* g_full_host);
int dq_codec_round_host(dq_ctx* ctx, const float* v_host, uint32_t round, float eta,
                        uint8_t* codes_x_host, float* delta_x_host, void* stream);

/* Dense quantise + pack WITHOUT a context and without any allocation.  The paper has no counterpart: this
 * entry point exists for callers that must not allocate device memory at the time of the call -- code running
 * inside another framework's memory pool or allocator callback, a process whose device memory is fully
 * budgeted up front, or a plug-in that is handed buffers and a stream and nothing else.  dq_create would call
 * cudaMalloc for its scratch; here the only scratch the dense path needs (one norm word per message) lives in
 * a fixed device array inside the library, which every GPU that loads the library holds until exit (about
 * 4 KiB).  It computes exactly what dq_quantize_sparsify_pack computes for sparsify = 0 with the same
 * (seed, round): v [M][d] -> codes [M][stride] packed b-bit codes and scale [M] = delta.
 *   - M may not exceed DQ_STATIC_MAX_MESSAGES; larger M returns DQ_ERR_SHAPE.  b must be 2, 4 or 8
 *     (DQ_ERR_BITS); stride >= dq_packed_bytes(d, b) and a multiple of 16; codes 16-byte aligned.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress) with that
 *     device current; make that first call outside any stream capture.  No call allocates or frees.
 *   - All calls on a device share the one array, which still holds the previous call's norms; each call
 *     clears what it needs on `stream` first.  Two calls whose GPU work overlaps (different streams, or
 *     different threads) race on it: serialise them.
 *   - A message that holds a NaN or an Inf gets scale 0 and all-zero codes (every coordinate, the non-finite ones
 *     included); there is no status word to poll.  scale must be 4-byte aligned.
 *   - The first call on a device may be made from several host threads at once.  The return value reports this call's
 *     own launches only. */
#define DQ_STATIC_MAX_MESSAGES 1024
int dq_quantize_pack_static(const float* v, int64_t d, int M, int b, uint64_t seed, uint32_t round,
                            uint8_t* codes, int64_t stride, float* scale, void* stream);

/* Test utility: dequantise message w of `msgs` into out [d] (zeros where a sparse message has no entry). */
int dq_unpack(dq_ctx* ctx, const dq_msgs* msgs, int w, float* out, void* stream);

/* Diagnostic: P(x) = f(x) + h(x) of eq. (1) over all n rows into one device double. */
int dq_objective(dq_ctx* ctx, const float* x, double* P, void* stream);

/* The context's own message buffers and last-round intermediates (device pointers, valid until
 * dq_destroy), for inspection after dq_round: alpha [M][d], norm_inf [M], batch rows [M][B]. */
int dq_round_buffers(dq_ctx* ctx, dq_msgs* msgs, const float** alpha, const float** norm_inf,
                     const int32_t** batch_idx, const uint8_t** codes_x, const float** delta_x);

/* Synchronises `stream`, returns the sticky device status through *status (HOST) and clears it. */
int dq_poll_status(dq_ctx* ctx, int* status, void* stream);

/* Number of kernels this context has launched so far (host counter). */
int64_t dq_launch_count(const dq_ctx* ctx);

const char* dq_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* DQ_H_ */
