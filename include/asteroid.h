/*
 * asteroid.h — C ABI of the per-stage micro-batched training step.
 *
 * A *stage* is a contiguous range of a network's layers; one *HPP-Round* on a stage is
 * FP over M micro-batches of size B, BP over the same micro-batches, accumulation of the
 * parameter gradients of all of them, and one update at the end (Asteroid, Section 3.2,
 * "HPP Architecture and Workflow").  The calls below are exactly those steps, plus the
 * per-layer profile that feeds the planner (Section 3.3, "DNN Model and Asteroid Profiler").
 *
 * Conventions
 *  - Every call returns 0 on success or a negative AST_ERR_* code; the text of the last error
 *    of the calling thread is available from asteroid_last_error().  Nothing throws or exits.
 *  - Activation tensors are DEVICE pointers, NHWC, in the stage's storage type (float or
 *    bfloat16), owned by the caller.  Parameter / state vectors passed to import/export are
 *    HOST pointers to float.  The stage owns its arenas and frees them in destroy.
 *  - `stream` is a cudaStream_t passed as void*.  forward/backward/accumulate/step and the loss
 *    heads only enqueue work on it; they never synchronise.  create, destroy, import, export
 *    and profile synchronise the device.  backward also enqueues the weight-gradient kernels on a
 *    stream of the stage that forks from `stream` and joins it before backward returns, so a whole
 *    round of these calls (after one plain round, in which first-use set-up happens) may be
 *    captured into a CUDA graph on `stream` and replayed.
 *  - The library has no CPU fallback: without a CUDA device every compute call fails.
 *
 * Flat parameter order (import/export): layers in list order; per layer
 *    conv    weight [c_out][k][k][c_in]
 *    dwconv  weight [c][k][k]
 *    bn      gamma [c], beta [c]
 *    linear  weight [c_out][c_in], bias [c_out]
 *    se      w1 [k][c], b1 [k], w2 [c][k], b2 [c]      (k = squeeze width)
 */
#ifndef ASTEROID_H
#define ASTEROID_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct asteroid_stage asteroid_stage;

enum { AST_CONV = 0, AST_DWCONV = 1, AST_BN = 2, AST_RELU6 = 3, AST_RELU = 4, AST_ADD = 5, AST_GAP = 6, AST_LINEAR = 7, AST_SILU = 8, AST_SE = 9 };
enum { AST_F32 = 0, AST_BF16 = 1 };
enum {
    AST_OK = 0,
    AST_ERR_ARG = -1,          /* null pointer, bad range, bad size */
    AST_ERR_UNSUPPORTED = -2,  /* a layer pattern or shape the kernels do not cover */
    AST_ERR_ORDER = -3,        /* call sequence violates the round (see each call) */
    AST_ERR_ALLOC = -4,        /* device allocation failed */
    AST_ERR_CUDA = -5,         /* a CUDA runtime call failed; text in asteroid_last_error() */
    AST_ERR_TIMEOUT = -6       /* a bounded device-side wait expired */
};

/* One layer of the network's layer sequence (Section 3.3: the model graph is topologically
 * sorted into a sequence of layers).  `src` is the index of the layer whose output this layer
 * reads, `add_from` (AST_ADD only) the index of the second operand; index -1 is the network
 * input.  Inside a stage [first,last] an index equal to first-1 denotes the stage input;
 * smaller indices are rejected.  Conv: cross-correlation, zero padding `pad`, no bias, weights
 * [c_out][k][k][c_in].  Dwconv: k = 3, 5 or 7, pad = (k-1)/2, c_in==c_out.  BN: training mode, statistics over
 * the micro-batch.  Add: out = value[src] + value[add_from].  ReLU6 / ReLU directly after a conv (or its BN) are applied
 * while the next layer loads; SiLU (x * sigmoid(x)) and SE are layers of their own whose output is stored.
 * SE (squeeze-excite of the EfficientNet block, one of the paper's vision workloads, Section 5.1), c_in == c_out == c,
 * `k` = squeeze width: s = mean over h,w; h = silu(w1 s + b1); g = sigmoid(w2 h + b2); out = x * g per sample and channel. */
typedef struct {
    int32_t op, c_in, c_out, k, stride, pad, src, add_from;
} ast_layer;

typedef struct {
    int32_t dtype;            /* AST_F32, or AST_BF16 = bfloat16 activations and activation gradients,
                                 float master weights, statistics, gradients and optimizer state */
    int32_t slots;            /* K: micro-batches that may be resident between their FP and BP
                                 (Section 3.2, K_p warm-up forwards); 0 means M */
    int32_t need_input_grad;  /* 0 for the first stage of a network: BP writes no dx */
    float bn_eps;             /* 0 means 1e-5 */
    float bn_momentum;        /* running-statistics momentum; 0 means 0.1 */
} ast_opts;

/* Per-layer record for the planner (Section 3.3): t_f, t_b at the given batch size, output
 * bytes a_l, weight bytes w_l; FLOPs as used by the re-planning of Section 3.4; and the three
 * memory terms of Eq. (3). */
typedef struct {
    double t_f_ms, t_b_ms;       /* median device time of the kernels that execute this layer's FP / BP.
                                    A layer fused into a neighbour's kernel reports 0 and names that
                                    neighbour in fused_into. */
    uint64_t a_l_bytes;          /* output activation bytes at `batch` in the storage type */
    uint64_t w_l_bytes;          /* float32 parameter bytes */
    uint64_t flops;              /* forward FLOPs at `batch`: 2 per multiply-accumulate of conv / linear layers */
    uint64_t alg_bytes_f;        /* bytes the layer's FP kernels must move (each tensor once) */
    uint64_t alg_bytes_b;        /* same for BP */
    uint64_t mem_mod;            /* Eq. (3) Mem_MOD: parameters, accumulated and per-micro-batch gradients, derived weight copies */
    uint64_t mem_opt;            /* Eq. (3) Mem_OPT: momentum */
    uint64_t mem_act;            /* Eq. (3) Mem_ACT(batch): one resident micro-batch's saved tensors */
    uint64_t mem_work;           /* BP workspace and reduction scratch (transient; not a term of Eq. (3)) */
    int32_t fused_into;          /* layer index whose kernels execute this layer, or -1 */
    int32_t reserved;
} ast_layer_profile;

/* Build the stage for layers [first,last] of `net` (Section 3.2: a stage model is a set of
 * consecutive layers), for micro-batches of `micro_batch` samples of in_h x in_w x net[first].c_in,
 * M micro-batches per round.  Parameters start at zero (gamma too): call import_state.
 * Errors: AST_ERR_ARG (range, sizes, references below first-1), AST_ERR_UNSUPPORTED (a BN or
 * activation that does not follow a conv/add it can fuse with, an intermediate of a fused
 * conv-BN-activation chain read by another layer, dwconv with k!=3), AST_ERR_ALLOC. */
int asteroid_stage_create(const ast_layer* net, int n_layers, int first, int last,
                          int in_h, int in_w, int micro_batch, int M,
                          const ast_opts* opts, asteroid_stage** out);
void asteroid_stage_destroy(asteroid_stage* s);

size_t asteroid_stage_param_count(const asteroid_stage* s);
/* Elements of the stage output per micro-batch, and its (h, w, c). */
size_t asteroid_stage_output_elems(const asteroid_stage* s, int* h, int* w, int* c);

/* Load parameters (and optionally momentum; NULL keeps/clears it to zero) from HOST memory;
 * n must equal param_count.  Also refreshes the derived weight copies the kernels read. */
int asteroid_stage_import_state(asteroid_stage* s, const float* params, const float* momentum, size_t n);
/* Copy state to HOST memory; any pointer may be NULL.  micro_grad is g_m of the last backward. */
int asteroid_stage_export_state(asteroid_stage* s, float* params, float* momentum, float* grad_accum,
                                float* micro_grad, size_t n);
/* BatchNorm running mean / variance (momentum update once per forward, unbiased variance),
 * concatenated over the stage's BN layers in layer order; n = sum of their channel counts. */
int asteroid_stage_export_bn_running(asteroid_stage* s, float* mean, float* var, size_t n);

/* FP of micro-batch `mb` (Section 3.2): reads x (B x in_h x in_w x c_in), writes the stage output y,
 * and keeps in an activation slot what BP of `mb` needs (x itself is copied, the caller may reuse
 * it).  Errors: AST_ERR_ARG (mb outside [0,M)), AST_ERR_ORDER (mb already resident, or `slots`
 * micro-batches already resident). */
int asteroid_stage_forward(asteroid_stage* s, int mb, const void* x, void* y, void* stream);
/* BP of micro-batch `mb`: reads dy = dL/dy, writes dx = dL/dx (ignored when need_input_grad==0) and the
 * parameter gradients g_mb of this micro-batch, then releases the slot.  The weight-gradient kernels,
 * on which nothing else in the pass depends, run on a stream the stage owns, forked from `stream`
 * after the coefficients they need and joined back into `stream` before the call returns: in
 * `stream` order the call is complete like any other.  Errors: AST_ERR_ORDER (no resident FP of mb,
 * or the previous g not yet accumulated). */
int asteroid_stage_backward(asteroid_stage* s, int mb, const void* dy, void* dx, void* stream);
/* G += g_mb: accumulate the gradients of the micro-batch whose BP ran last (Section 3.2: each device
 * accumulates gradients for all micro-batches of the mini-batch).  AST_ERR_ORDER if mb is not that one. */
int asteroid_stage_accumulate(asteroid_stage* s, int mb, void* stream);
/* Accumulated-gradient arena of the stage, for the gradient synchronisation of a data-parallel device group
 * (Section 3.2: the devices of a group hold replicas of the stage, each runs its share of every micro-batch and
 * the gradients are synchronised with an AllReduce before the update; Eq. (5) counts its volume).  *G receives a
 * DEVICE pointer to the float32 arena that asteroid_stage_accumulate adds into and asteroid_stage_step consumes,
 * *n its length in floats (parameters in layer order, every layer starting at a multiple of 8 floats, the
 * padding is zero).  The stage owns the memory; the pointer stays valid until asteroid_stage_destroy.  Between the
 * last accumulate of a round and asteroid_stage_step a group member may scale the arena by its share of the
 * micro-batch (y_d / B) and sum it over the group on the stream its stage calls use; the library itself does no
 * communication.  AST_ERR_ARG for a null argument. */
int asteroid_stage_grad_buffer(asteroid_stage* s, float** G, size_t* n);
/* End of the HPP-Round (Section 3.2: accumulated gradients are applied to the stage parameters):
 * g = G/M; v = momentum*v + g; w = w - lr*v; G = 0; derived weight copies refreshed.
 * AST_ERR_ORDER unless exactly M micro-batches were accumulated since the last step. */
int asteroid_stage_step(asteroid_stage* s, float lr, float momentum, void* stream);

/* Per-layer cost record at batch size `batch` (Section 3.3: FP/BP time of each layer for various
 * batch sizes, output size and weight size in bytes).  Runs the stage's own kernels on zero-filled
 * buffers of that batch size (3 warm-up + 7 timed rounds, CUDA events), synchronises.
 * `layer` is an index in [first,last].  The timed launch plan is the one a round uses (BatchNorm
 * statistics and backward sums taken inside the neighbouring kernels wherever the round does so),
 * except that every kernel stays on one stream, so that a layer's time is that of its own kernels.
 * A BatchNorm whose sums were taken by another layer's kernel reports only its finishing kernel
 * (alg_bytes of a few kB, or 0) and names that layer in fused_into. */
int asteroid_stage_profile(asteroid_stage* s, int layer, int batch, ast_layer_profile* out);

/* Loss heads (used by the last stage and by tests).  All pointers are DEVICE pointers.
 * MSE: *loss = mean((y-t)^2) over n elements, dy = 2 (y-t) / n. */
int asteroid_loss_mse(const void* y, const void* target, size_t n, int dtype, void* dy, float* loss, void* stream);
/* The same MSE head for callers that must not allocate device memory (the paper has no counterpart;
 * this serves hosts that run the round inside a fixed memory budget, a memory pool that forbids
 * cudaMalloc after start-up, or a region where allocation is illegal).  asteroid_loss_mse obtains
 * its reduction scratch with cudaMalloc on first use; this variant keeps the scratch (4.25 KB: one
 * partial sum per block and a ticket word) in a static device array inside the library, which every
 * GPU context that loads the library holds until the process exits.  It never calls cudaMalloc,
 * cudaFree or any allocating routine.
 *  - n must not exceed 67 108 864 elements (AST_ERR_ARG with a message otherwise).
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress) with
 *    that device current; make that first call before starting any stream capture.
 *  - All calls on a device share the one array: each call clears the ticket word on `stream` before
 *    its kernel, and two calls whose kernels may overlap on the GPU (different streams) race.
 *  - Concurrent first calls on one device from several host threads are safe (each stores the same address).
 *    Device ordinals of 64 and above are refused with AST_ERR_ARG. */
int asteroid_loss_mse_noalloc(const void* y, const void* target, size_t n, int dtype, void* dy, float* loss, void* stream);
/* Softmax cross-entropy: *loss = mean_r(-log softmax(logits_r)[labels_r]),
 * dlogits = (softmax - onehot) / rows.  rows <= 65536. */
int asteroid_loss_softmax_xent(const void* logits, const int32_t* labels, int rows, int classes, int dtype,
                               void* dlogits, float* loss, void* stream);

/* Kernel-level trace (the paper has no counterpart; its profiler works per layer, Section 3.3).
 * Between start and stop every kernel launch of the library is bracketed by CUDA events on its
 * stream; stop synchronises the device and returns, per kernel kind that ran, the number of
 * launches, the summed device time, the summed algorithmic bytes (each tensor the kernel must
 * read or write, once) and floating-point operations.  At most `capacity` records are written,
 * *n_out receives the count.  Tracing adds two event records per launch and keeps every kernel on the
 * caller's stream (no overlap with the stage's second stream), so that a recorded duration is that of
 * the kernel running alone: do not time throughput while it is on. */
typedef struct {
    char name[48];
    uint64_t launches;
    double total_ms, alg_bytes, flops;
} ast_kernel_stat;
int asteroid_trace_start(void);
int asteroid_trace_stop(ast_kernel_stat* out, int capacity, int* n_out);

/* ---- Parallelism planning (Section 3.3, "Parallelism Planning"), host only --------------------------------------------
 * Input: the profiler's cost tables per device type (FP / BP milliseconds of every layer at the profiled batch sizes;
 * times between profiled sizes are interpolated linearly, 0 at batch 0, the last segment continued beyond the largest),
 * per layer the output bytes per sample a_l, the parameter bytes w_l and the bytes kept per sample for BP; the device
 * pool (type and memory budget of each device, pairwise bandwidth in bytes per millisecond); micro-batch size B,
 * micro-batches per round M, and the block of samples the offloading phase moves at a time.
 * All pointers are HOST pointers owned by the caller.  Layouts: t_f, t_b [n_types][L][n_bs]; bw [N][N].
 * Memory of a device holding layers i..j with y samples as the stage K-th from the end (Eq. (3)):
 *     (mod_factor + opt_factor) * sum w_l + (2K - 1) * y * sum act_l  <=  dev_mem.                                  */
#define AST_PLAN_MAX_DEVICES 64
typedef struct {
    int32_t L, n_types, n_bs, N, B, M, block;
    const int32_t* bs;
    const double *t_f, *t_b;
    const double *a, *w, *act;
    double mod_factor, opt_factor;
    const int32_t* dev_type;
    const double* dev_mem;
    const double* bw;
} ast_plan_problem;

/* The chosen hybrid pipeline: n_stages stages in pipeline order; stage s runs layers first_layer[s]..last_layer[s]
 * data-parallel on devices[dev_begin[s] .. dev_begin[s+1]) (indices into the caller's device arrays), device
 * devices[q] taking samples[q] of every micro-batch.  e_f/e_b/t_a: FP, BP and AllReduce milliseconds of the stage
 * (Eq. (5), (8)); dominant_step indexes the step list exec, comm, exec, ... (Eq. (11)); latency_ms is the estimated
 * HPP-Round latency (Eq. (4)).  n_stages == 0 with infinite latency: no configuration fits the memory budgets. */
typedef struct {
    double latency_ms;
    int32_t n_stages, n_steps, dominant_step, reserved;
    int32_t first_layer[AST_PLAN_MAX_DEVICES], last_layer[AST_PLAN_MAX_DEVICES], dev_begin[AST_PLAN_MAX_DEVICES + 1];
    int32_t devices[AST_PLAN_MAX_DEVICES], samples[AST_PLAN_MAX_DEVICES];
    double e_f_ms[AST_PLAN_MAX_DEVICES], e_b_ms[AST_PLAN_MAX_DEVICES], t_a_ms[AST_PLAN_MAX_DEVICES];
} ast_plan_result;

/* Algorithm 2 (dynamic programming over layers, devices in descending order of memory, and stage count; Eq. (10)) with
 * Algorithm 1 (memory-aware balancing, then straggler offloading; Eq. (7)-(9)) for every candidate stage.
 * Errors: AST_ERR_ARG (null table, non-positive size, more than 64 devices, batch sizes not ascending, bad device type). */
int asteroid_plan(const ast_plan_problem* problem, ast_plan_result* result);

/* Self-test of the bounded device-side waits (the paper has no counterpart).  Every hand-off wait inside the
 * tensor-core kernels gives up after a fixed number of polls, sets the stage's error word and lets the kernel
 * return, which export_state then reports as AST_ERR_TIMEOUT.  This call runs that mechanism on purpose: one
 * warp waits 1024 polls on a barrier at which nobody arrives.  Returns AST_ERR_TIMEOUT when the wait gave up and
 * the kernel returned (the expected outcome), AST_OK if the wait reported success, AST_ERR_CUDA on a runtime
 * error.  Synchronises the device; the context stays usable. */
int asteroid_selftest_bounded_wait(void);

/* Count of kernel launches this library has enqueued in the calling process. */
uint64_t asteroid_launch_count(void);
const char* asteroid_last_error(void);

#ifdef __cplusplus
}
#endif
#endif
