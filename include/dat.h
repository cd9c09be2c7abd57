/*
 * dat.h -- C ABI of the B200 (sm_100a) implementation of the data-parallel hot path of
 * the outer-minimisation step of Distributed Adversarial Training (DAT):
 *
 *     M workers' per-layer fp32 gradients
 *       -> randomized b-bit quantizer Q(.)              [Algorithm A1 Step 7; Eq. rand_q, Eq. xi]
 *       -> aggregation  g_hat = (1/M) sum_i Q(g^(i))    [Algorithm A1 Step 9; Eq. grad_agg]
 *       -> layer-wise adaptive learning-rate update      [Algorithm A1 Step 12, Eq. outer_min; Eq. 3]
 *
 * On one GPU the M workers are M gradient buffers in device memory.
 *
 * General conventions
 *   - Every function returns an int: DAT_OK (0) or a negative DAT_ERR_* code.  Nothing throws,
 *     aborts or prints.  Faults that the host can detect (null pointers, misalignment, bad
 *     sizes) are returned BEFORE any kernel is launched.
 *   - "device" pointers address memory of the CUDA device that was current when the plan was
 *     created; that device must also be current in every later call with the plan.
 *     "host" pointers address ordinary host memory.
 *   - The caller owns every data buffer.  The library never allocates, frees or retains them;
 *     after a call returns, only work already enqueued on `stream` refers to them.
 *     A plan owns only its own small device workspace (layout tables, partial sums,
 *     arrival counters, a status word) and, if dat_step_host is used, staging buffers.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All device work
 *     is enqueued on it and is stream-ordered; calls return without synchronising unless
 *     stated otherwise.
 *   - Device data pointers must be 16-byte aligned (DAT_ERR_ALIGN otherwise).  Layer offsets
 *     may be arbitrary (a layer need not start on a 16-byte boundary).
 *   - A plan must not be used from two host threads at once, nor by two calls that overlap on
 *     the device (its workspace is shared); distinct plans are independent.
 *   - Conditions only the device can see (non-finite inputs, a bounded wait that ran out) set
 *     bits in the plan's status word, read with dat_get_status; they never trap or hang.
 *
 * Notation: d = total number of parameters, h = number of layers (one per parameter tensor,
 * given by the offset table), n_l = elements of layer l, M = workers, b = bits,
 * S = 2^b - 1 (largest level), nu_l = the quantizer norm of layer l.
 */
#ifndef DAT_H_
#define DAT_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DAT_MAX_WORKERS 64

typedef struct dat_plan dat_plan_t;

/* Hyper-parameters of the update (Eq. 3): learning rate eta_t, momentum mu and weight decay of
 * the descent direction u = mu*m + g_hat + wd*theta, and the clamp tau(x) = min{max{x,c_l},c_u}
 * (the paper's experiments use c_l = 0, c_u = 10). */
typedef struct dat_hparams {
    float lr;
    float momentum;
    float weight_decay;
    float c_l;
    float c_u;
} dat_hparams_t;

/* Hyper-parameters of the LAMB direction (Algorithm A2) and of the update of Eq. upth: beta1, beta2
 * of the two moments (each in (0,1)), zeta > 0 of the ratio m^/(sqrt(v^) + zeta), weight decay (added
 * to the ratio as in the LAMB paper; 0 gives the algorithm as printed), and lr, c_l, c_u as above.
 * The paper's ImageNet runs use beta1 = 0.9, beta2 = 0.999, weight decay 1e-4. */
typedef struct dat_lamb_hparams {
    float lr;
    float beta1;
    float beta2;
    float zeta;
    float weight_decay;
    float c_l;
    float c_u;
} dat_lamb_hparams_t;

/* Which l2 norm scales the quantizer of Eq. rand_q.
 * SHARED_MAX: nu_l = max_i ||g_l^(i)||_2, one value per layer shared by all workers, so that
 *             the workers' integer codes lie on one grid and Eq. grad_agg becomes an integer sum
 *             followed by one scaling.  (Q stays unbiased for any nu >= max|g|.)
 * PER_WORKER: nu_{i,l} = ||g_l^(i)||_2, every worker's own norm, as Eq. rand_q and Eq. grad_agg
 *             are written: g_hat = (1/M) sum_i nu_{i,l} * sign * level / S, summed in fp32.  The
 *             message then carries M*h norms (index i*h + l), and no integer code sum exists.
 *             dat_step_passes, which sums integer codes, answers DAT_ERR_UNSUPPORTED for such a
 *             plan; every other call takes it.                                                  */
enum { DAT_SCALE_SHARED_MAX = 0, DAT_SCALE_PER_WORKER = 1 };

/* Resolution of the quantizer's uniform number (see dat_plan_create). */
enum { DAT_RNG_BITS_16 = 16, DAT_RNG_BITS_23 = 23 };

enum {
    DAT_OK = 0,
    DAT_ERR_ARG = -1,          /* null pointer, negative size, value out of range              */
    DAT_ERR_ALIGN = -2,        /* a device data pointer is not 16-byte aligned                 */
    DAT_ERR_BITS = -3,         /* bits not in {1,2,4,8,16,32}, or not valid for this call      */
    DAT_ERR_LAYOUT = -4,       /* offsets[0] != 0 or offsets not strictly increasing           */
    DAT_ERR_CUDA = -5,         /* a CUDA runtime call failed (see dat_last_cuda_error)         */
    DAT_ERR_NOMEM = -6,        /* host or device allocation failed                              */
    DAT_ERR_UNSUPPORTED = -7,  /* valid request that this build does not implement             */
    DAT_ERR_TOO_LARGE = -8     /* problem exceeds a fixed capacity (dat_lalr_step_static)       */
};

/* Bits of the device status word. */
enum {
    DAT_STATUS_NONFINITE = 1u, /* a quantizer norm or a layer norm was inf or NaN              */
    DAT_STATUS_TIMEOUT = 2u,   /* a bounded device-side wait ran out; outputs are undefined until
                                  dat_get_status has been called (which restores the plan)      */
    DAT_STATUS_BOUNDS = 4u     /* reserved for self-checking builds                             */
};

/* ---------------------------------------------------------------------------------------------
 * Plan: the layer partition theta = [theta_1^T ... theta_h^T]^T of Eq. 3 and the quantizer setup.
 *   out            host pointer receiving the new plan.
 *   num_layers     h >= 1.
 *   layer_offsets  host array of h+1 element offsets; offsets[0] = 0, strictly increasing,
 *                  offsets[h] = d.  Copied; the caller may free it after the call.
 *   num_workers    M in [1, DAT_MAX_WORKERS].
 *   bits           b in {1,2,4,8,16}, or 32 = no quantisation (Q is the identity and the
 *                  aggregate is the plain worker average).
 *   scale_mode     DAT_SCALE_SHARED_MAX or DAT_SCALE_PER_WORKER.
 *   rng_bits       resolution of the uniform number u of the stochastic rounding (Eq. xi; the
 *                  paper fixes neither generator nor resolution).  Randomness is Philox4x32-10
 *                  keyed on (seed, step, worker, element):
 *                  DAT_RNG_BITS_23: one block per four consecutive elements (counter
 *                    (lo(e/4), hi(e/4), worker, hi(seed)), key (lo(seed), step)), element e takes
 *                    word e mod 4, u = (low 23 bits) / 2^23;
 *                  DAT_RNG_BITS_16: one block per eight consecutive elements (counter e/8),
 *                    element e takes word (e/2) mod 4, low half if e is even, high half if odd,
 *                    u = half / 2^16.  Half the generator work per element; the rounding
 *                    probability matches frac(x) to 2^-16 of a level.
 *                  Ignored for bits = 32.
 * Allocates the plan's device workspace (synchronous).  Errors: ARG, BITS, LAYOUT, NOMEM, CUDA.
 * ------------------------------------------------------------------------------------------- */
int dat_plan_create(dat_plan_t **out, int64_t num_layers, const int64_t *layer_offsets,
                    int num_workers, int bits, int scale_mode, int rng_bits);

/* dat_plan_set_origin -- for a plan that covers a SLICE of a larger problem (a contiguous range of layers
 * and a subset of the workers, as one rank of a sharded step holds them): the global index of the plan's
 * element 0 (a multiple of 8) and of its worker 0.  dat_quantize and dat_requantize then draw exactly the
 * random numbers the unsliced problem would draw for those elements and workers (the paper's Q is keyed on
 * (seed, step, worker, element) here).  dat_step and dat_step_passes answer DAT_ERR_UNSUPPORTED for a plan
 * with a non-zero origin.  Errors: ARG. */
int dat_plan_set_origin(dat_plan_t *plan, int64_t elem_base, int64_t worker_base);

/* Frees the plan and its workspace (synchronises the device).  NULL is accepted. */
int dat_plan_destroy(dat_plan_t *plan);

/* Sizes of the caller-owned buffers of the unfused calls (any output pointer may be NULL):
 *   level_bytes_per_worker  bytes of one worker's level plane: ceil(d*b/8) rounded up to 16
 *   sign_bytes_per_worker   bytes of one worker's sign plane:  ceil(d/8)   rounded up to 16
 *   num_scales              number of fp32 norms in the message (h; M*h with per-worker scales)
 *   workspace_bytes         device bytes the plan itself holds
 * Together: 32 bits per norm + d sign bits + b*d level bits per worker -- the
 * "(32 + d + b d) bits" message of the paper's quantizer, with one norm per layer.            */
int dat_plan_sizes(const dat_plan_t *plan, int64_t *level_bytes_per_worker,
                   int64_t *sign_bytes_per_worker, int64_t *num_scales, int64_t *workspace_bytes);

/* ---------------------------------------------------------------------------------------------
 * dat_quantize -- Algorithm A1 Step 7: Q(g^(i)) for every worker (Eq. rand_q, Eq. xi).
 *   For worker i, layer l, element e (global index in the flat vector), with x = S*|g_e|/nu_l:
 *   level = floor(x) + 1 with probability x - floor(x), else floor(x); sign bit = (g_e < 0).
 *   Randomness: Philox4x32-10 keyed on (seed, step, worker i, element e); u1 = 1 + u with u the
 *   plan's 23-bit or 16-bit uniform number (see rng_bits of dat_plan_create);
 *   level = min(floor(fma(|g_e|, S/nu_l, u1)) - 1, S).
 *
 *   grads      host array of M device pointers, each fp32[d], read-only.
 *   seed,step  random-stream key; step must be < 2^32 (DAT_ERR_ARG).
 *   levels     device, M * level_bytes_per_worker bytes, written.  Worker i's plane starts at
 *              i*level_bytes_per_worker.  A plane is a little-endian bit stream over the global
 *              element index: element e occupies bits [(e*b) mod 8, +b) of byte floor(e*b/8)
 *              (b = 16: a little-endian uint16).  Padding bytes are written as zero.
 *   signs      device, M * sign_bytes_per_worker bytes, written: bit (e mod 8) of byte
 *              floor(e/8), 1 = negative.
 *   scales     device fp32[num_scales], written: nu_l (per-worker scales: nu_{i,l} at i*h + l).
 *   scales_in  device fp32[num_scales] or NULL.  If given, these norms are used instead of computing
 *              ||g_l^(i)||_2 (and are copied to `scales`); may alias `scales`.
 * Errors: ARG, ALIGN, BITS (b = 32 has no codes), CUDA.
 * ------------------------------------------------------------------------------------------- */
int dat_quantize(dat_plan_t *plan, const float *const *grads, uint64_t seed, uint64_t step,
                 uint8_t *levels, uint8_t *signs, float *scales, const float *scales_in,
                 void *stream);

/* dat_worker_norms -- the norms of Eq. rand_q by themselves: nu_{i,l} = ||g_l^(i)||_2 for every worker and
 * layer (fp64 sums of exact squares, one rounding), without drawing any level.  A sharded step needs them
 * before it can agree on the shared norm max_i nu_{i,l} across ranks.
 *   grads      host array of M device pointers, fp32[d] each, read-only.
 *   norms_out  device fp32[M*h], written: nu_{i,l} at i*h + l.
 * Errors: ARG, ALIGN, CUDA. */
int dat_worker_norms(dat_plan_t *plan, const float *const *grads, float *norms_out, void *stream);

/* ---------------------------------------------------------------------------------------------
 * dat_aggregate -- Algorithm A1 Step 9, Eq. grad_agg, on the packed messages:
 *   sum_e = sum_i (sign ? -level : level)  (exact, int32);  g_hat_e = sum_e * (nu_l / (S*M)).
 *   levels, signs, scales   device, as written by dat_quantize, read-only.
 *   code_sum                device int32[d] or NULL; written if given.  With per-worker scales
 *                           g_hat_e = (sum_i fma(nu_{i,l}, signed level_i, .)) / (S*M) in ascending
 *                           worker order, and code_sum must be NULL (DAT_ERR_ARG).
 *   g_hat                   device fp32[d], written.
 * Errors: ARG, ALIGN, BITS (b = 32), CUDA.
 * ------------------------------------------------------------------------------------------- */
int dat_aggregate(dat_plan_t *plan, const uint8_t *levels, const uint8_t *signs,
                  const float *scales, int32_t *code_sum, float *g_hat, void *stream);

/* dat_aggregate_gather -- dat_aggregate with one pointer per worker instead of one buffer: worker i's level
 * plane at level_planes[i] (level_bytes_per_worker bytes) and sign plane at sign_planes[i].  The planes may lie
 * in this GPU's memory or in a peer GPU's memory that is mapped into the process (peer access, an IPC or
 * symmetric-memory mapping): the kernel reads them with plain loads, so the owner of a layer range of a sharded
 * step pulls the other ranks' messages over NVLink while it sums them -- exchange and Step 9 in one kernel.
 * The caller guarantees that the planes are complete before the call's work starts (a barrier between the
 * ranks) and are not rewritten before it ends.
 *   level_planes, sign_planes   host arrays of M device pointers, each 16-byte aligned, read-only.
 * Other arguments, results (bit for bit) and errors as dat_aggregate. */
int dat_aggregate_gather(dat_plan_t *plan, const uint8_t *const *level_planes, const uint8_t *const *sign_planes,
                         const float *scales, int32_t *code_sum, float *g_hat, void *stream);

/* ---------------------------------------------------------------------------------------------
 * dat_requantize -- Algorithm A1 Step 10 (two-sided quantisation, the parameter-server setting):
 * the server quantizes the aggregate once more before sending it back, g_hat <- Q(g_hat).
 *   Q is the quantizer of dat_quantize applied to ONE vector: nu_l = ||g_hat_l||_2 (or
 *   scales_in[l]), random stream of index M (the first one no worker uses; the paper does not say
 *   where the server's random numbers come from), level = min(floor(fma(|g|, S/nu_l, u1)) - 1, S),
 *   and the receiver's value nu_l * sign * level / S, which overwrites g_hat.
 *   g_hat      device fp32[d], read and overwritten.
 *   levels     device, level_bytes_per_worker bytes, written: the server's level plane.
 *   signs      device, sign_bytes_per_worker bytes, written.
 *   scales     device fp32[h], written: nu_l.       scales_in  device fp32[h] or NULL, as in dat_quantize.
 * Valid for any plan with b < 32, whatever its scale mode.  Errors: ARG, ALIGN, BITS, CUDA.
 * ------------------------------------------------------------------------------------------- */
int dat_requantize(dat_plan_t *plan, float *g_hat, uint64_t seed, uint64_t step, uint8_t *levels,
                   uint8_t *signs, float *scales, const float *scales_in, void *stream);

/* dat_average -- Eq. grad_agg when Q is the identity (b = 32): g_hat_e = (sum_i g_e^(i)) / M,
 * accumulated in fp32 in ascending worker order.  Valid for any plan.
 *   grads  host array of M device pointers (fp32[d], read-only);  g_hat  device fp32[d], written. */
int dat_average(dat_plan_t *plan, const float *const *grads, float *g_hat, void *stream);

/* ---------------------------------------------------------------------------------------------
 * dat_lalr_step -- Algorithm A1 Step 12 with the LALR rule of Eq. 3, for every layer l:
 *   m'     = mu*m + (g_hat + wd*theta)                       (descent direction u = m')
 *   theta' = theta - tau(||theta_l||_2) * lr / ||u_l||_2 * u,  tau(x) = min{max{x,c_l},c_u}
 *   (||theta_l|| is the norm BEFORE the update; ||u_l|| = 0 gives a zero step.)
 *   Two passes: pass 1 writes m' and reduces the two norms per layer, pass 2 updates theta.
 *   theta, mom        device fp32[d], updated in place.
 *   g_hat             device fp32[d], read-only.
 *   hp                host pointer, read during the call.
 *   layer_norms_out   device fp32[2h] or NULL: [2l] = ||theta_l||, [2l+1] = ||u_l||.
 * Errors: ARG, ALIGN, CUDA.
 * ------------------------------------------------------------------------------------------- */
int dat_lalr_step(dat_plan_t *plan, float *theta, float *mom, const float *g_hat,
                  const dat_hparams_t *hp, float *layer_norms_out, void *stream);

/* ---------------------------------------------------------------------------------------------
 * dat_lamb_step -- Algorithm A1 Step 12 with LAMB (Algorithm A2) as the outer-minimisation oracle.
 * Per element (fp32, one rounding per operation), with t >= 1 the iteration count:
 *   m' = fma(beta1, m, (1-beta1)*g_hat)     v' = fma(beta2, v, (1-beta2)*(g_hat*g_hat))
 *   m^ = m'/(1-beta1^t)     v^ = v'/(1-beta2^t)     u = fma(wd, theta, m^/(sqrt(v^) + zeta))
 * and per layer (Eq. upth): theta' = theta - lr*tau(||theta_l||)/||u_l|| * u, norms in fp64, zero
 * norms as in dat_lalr_step.  The bias-corrected moments are temporaries; m', v' are what is stored.
 *   theta, mom, var  device fp32[d], updated in place.     g_hat  device fp32[d], read-only.
 *   layer_norms_out  device fp32[2h] or NULL: (||theta_l||, ||u_l||).
 * Errors: ARG (null pointer, t < 1, beta outside (0,1)), ALIGN, CUDA.
 * ------------------------------------------------------------------------------------------- */
int dat_lamb_step(dat_plan_t *plan, float *theta, float *mom, float *var, const float *g_hat,
                  const dat_lamb_hparams_t *hp, int64_t t, float *layer_norms_out, void *stream);

/* ---------------------------------------------------------------------------------------------
 * dat_lalr_step_static -- the update of dat_lalr_step for callers that must not allocate.
 * (The paper has no counterpart; this is a deployment variant of the same arithmetic.)
 *
 * Who needs it: code that runs where device allocation is forbidden or impossible -- inside a
 * framework's own allocator callbacks or a memory-pool's critical section, in a process whose
 * device memory was handed out completely at start-up, or in a host thread that is not allowed
 * to take the driver's allocation lock (a latency-critical serving loop).  Creating a plan
 * calls cudaMalloc; this entry point needs no plan and calls no cudaMalloc, cudaFree or any
 * other allocating routine.  Its scratch memory (the layer table, two fp64 partial sums per
 * 4096-element tile, one step length per layer; about 0.6 MB) is a fixed array inside the
 * library image, so every GPU that loads the library holds it until the process exits.
 *
 *   num_layers      h, 1 <= h <= DAT_STATIC_MAX_LAYERS.
 *   layer_offsets   HOST array of h+1 element offsets (as for dat_plan_create); copied during
 *                   the call.  The layers may span at most DAT_STATIC_MAX_TILES tiles of 4096
 *                   elements (each layer occupies ceil((n_l + 3)/4096) or fewer); larger
 *                   problems are refused with DAT_ERR_TOO_LARGE before anything is launched.
 *   theta, mom      device fp32[d], updated in place.      g_hat  device fp32[d], read-only.
 *   hp              host pointer, read during the call.
 *   layer_norms_out device fp32[2h] or NULL, as in dat_lalr_step.
 * The result is bit-identical to dat_lalr_step on the same inputs.
 * First call on a device: it looks up the device address of the scratch array (once per device,
 * with that device current).  The call copies its layer table from host memory on every call, so it
 * cannot be recorded into a CUDA graph: while `stream` is capturing it answers DAT_ERR_UNSUPPORTED
 * and enqueues nothing.  The call is not thread-safe with respect to other first calls on the same
 * device, and the looked-up address does not survive a cudaDeviceReset of that device.
 * All calls on a device share the one scratch array, which keeps the previous call's contents;
 * the call clears what has to start at zero.  Two calls whose device work overlaps (different
 * streams, or different host threads) race on it: serialise them.  Non-finite norms are not
 * reported (there is no plan whose status word could carry the bit).
 * Errors: ARG, ALIGN, LAYOUT, TOO_LARGE, UNSUPPORTED (device ordinal >= 64, or `stream` is capturing), CUDA.
 * ------------------------------------------------------------------------------------------- */
#define DAT_STATIC_MAX_LAYERS 4096
#define DAT_STATIC_MAX_TILES 32768
int dat_lalr_step_static(int64_t num_layers, const int64_t *layer_offsets, float *theta, float *mom,
                         const float *g_hat, const dat_hparams_t *hp, float *layer_norms_out, void *stream);

/* ---------------------------------------------------------------------------------------------
 * dat_step -- Steps 7, 9 and 12 of Algorithm A1 in one call: the result equals
 * dat_quantize -> dat_aggregate -> dat_lalr_step (or dat_average -> dat_lalr_step when b = 32),
 * but codes, code sums and g_hat are never written to device memory.  One kernel launch
 * (dat_step_pipelined); nothing is allocated and nothing synchronises: every table the launch
 * needs was built by dat_plan_create.
 *   theta, mom        device fp32[d], updated in place.
 *   grads             host array of M device pointers, fp32[d] each, read-only.
 *   seed, step        as in dat_quantize.
 *   hp                host pointer, read during the call.
 *   code_sum_out      device int32[d] or NULL (checking aid; ignored when b = 32).
 *   layer_norms_out   device fp32[2h] or NULL.
 *   scales_out        device fp32[h] or NULL: nu_l (not written when b = 32).
 * Inside the launch a work item may have to wait for a layer's norm that another item is still
 * producing; that wait is bounded (about two seconds).  If it ever runs out, the call returns as
 * usual, DAT_STATUS_TIMEOUT is set in the status word, and the outputs of that call -- and of
 * later calls on the plan -- are undefined until dat_get_status has been called, which reports the
 * bit and restores the plan's counters.
 * The call cannot be recorded into a CUDA graph (its epoch and the key of its random streams are launch
 * parameters, which a replay would repeat): while `stream` is capturing it answers DAT_ERR_UNSUPPORTED and
 * enqueues nothing.  The same holds for dat_step_lamb, dat_step_two_sided and dat_step_lamb_two_sided.
 * With a DAT_SCALE_PER_WORKER plan the step follows Eq. grad_agg as written (every worker on its own grid,
 * fp32 sum in ascending worker order): scales_out then has M*h entries (index i*h + l) and code_sum_out is
 * ignored (no integer sums exist).
 * Errors: ARG, ALIGN, UNSUPPORTED (plan with an origin; capturing stream), CUDA.
 * ------------------------------------------------------------------------------------------- */
int dat_step(dat_plan_t *plan, float *theta, float *mom, const float *const *grads,
             uint64_t seed, uint64_t step, const dat_hparams_t *hp,
             int32_t *code_sum_out, float *layer_norms_out, float *scales_out, void *stream);

/* dat_step_pipelined -- what dat_step calls: the step as ONE launch of ordinary thread blocks.  The
 * vector is cut into per-layer tiles; a work item holds one tile for each of three phases -- sums of
 * squares for the quantizer norms (N), levels + signed sum + g_hat + m' + layer sums (Q), parameter
 * update (U) -- with the Q tiles running a fixed distance behind the N tiles and the U tiles behind the
 * Q tiles, far enough that a part seldom has to wait for the layer-wide result it needs.  The gradients are
 * read twice (norm, then levels; from the L2 cache the second time only for small layers); codes, sums and
 * g_hat stay in registers.
 * Same arguments, results and errors as dat_step. */
int dat_step_pipelined(dat_plan_t *plan, float *theta, float *mom, const float *const *grads,
                       uint64_t seed, uint64_t step, const dat_hparams_t *hp, int32_t *code_sum_out,
                       float *layer_norms_out, float *scales_out, void *stream);

/* dat_step_lamb -- dat_step with LAMB (Algorithm A2) as the outer-minimisation oracle instead of the momentum
 * direction: Steps 7 and 9 as in dat_step, then m', v', the bias-corrected direction and the layer-wise update
 * exactly as dat_lamb_step computes them from g_hat -- in the same single launch, g_hat never stored.
 *   var   device fp32[d], the second moment, updated in place;  t >= 1 the iteration count;  hp as in dat_lamb_step.
 * Other arguments, the bounded wait and its status bit as in dat_step.
 * Errors: ARG (null pointer, t < 1, beta outside (0,1)), ALIGN, CUDA. */
int dat_step_lamb(dat_plan_t *plan, float *theta, float *mom, float *var, const float *const *grads,
                  uint64_t seed, uint64_t step, const dat_lamb_hparams_t *hp, int64_t t,
                  int32_t *code_sum_out, float *layer_norms_out, float *scales_out, void *stream);

/* dat_step_two_sided -- dat_step with two-sided quantisation (Algorithm A1 Step 10, the parameter-server
 * setting): after Steps 7 and 9 the server quantizes the aggregate itself, g_hat <- Q(g_hat), with its own
 * norm nu^_l = ||g_hat_l||_2 per layer and the levels of Eq. xi drawn on the random stream of index M (the
 * first one no worker uses) -- what dat_requantize computes -- and Step 12 uses the receiver's value.  All in
 * the same single launch: a fourth stream of tiles runs between the Q and the U tiles, waiting (bounded, as
 * in dat_step) for the layer's nu^_l.  Neither the workers' nor the server's packed message is written.
 *   g_hat               device fp32[d], caller-owned, 16-byte aligned: workspace (the aggregate is stored
 *                       here between the two phases) and output: on return the receiver's value
 *                       nu^_l * sign * level / S of every element.
 *   server_scales_out   device fp32[h] or NULL: nu^_l.
 * Other arguments, the bounded wait and its status bit as in dat_step; shared or per-worker plans.
 * Errors: ARG, ALIGN, BITS (b = 32: nothing to quantize with), UNSUPPORTED (plan with an origin), CUDA. */
int dat_step_two_sided(dat_plan_t *plan, float *theta, float *mom, const float *const *grads,
                       uint64_t seed, uint64_t step, const dat_hparams_t *hp, float *g_hat,
                       int32_t *code_sum_out, float *layer_norms_out, float *scales_out,
                       float *server_scales_out, void *stream);

/* dat_step_lamb_two_sided -- dat_step_lamb with Step 10 between the aggregation and Algorithm A2, as in
 * dat_step_two_sided (same g_hat and server_scales_out). */
int dat_step_lamb_two_sided(dat_plan_t *plan, float *theta, float *mom, float *var, const float *const *grads,
                            uint64_t seed, uint64_t step, const dat_lamb_hparams_t *hp, int64_t t, float *g_hat,
                            int32_t *code_sum_out, float *layer_norms_out, float *scales_out,
                            float *server_scales_out, void *stream);

/* dat_step_passes -- the same step as dat_step, with the same arguments and the same results bit for
 * bit up to the norms' last place, computed by three streaming passes in separate launches: quantizer
 * norms; then levels, signed sum over the workers, g_hat, m' and the layer sums in one pass that keeps
 * codes, sums and g_hat in registers; then the theta update.  The gradients are read twice by
 * construction.  For plans with b < 32 and the shared scale (DAT_ERR_UNSUPPORTED otherwise).  Its first
 * call on a plan allocates two small tables (synchronous: not for use under stream capture). */
int dat_step_passes(dat_plan_t *plan, float *theta, float *mom, const float *const *grads,
                    uint64_t seed, uint64_t step, const dat_hparams_t *hp, int32_t *code_sum_out,
                    float *layer_norms_out, float *scales_out, void *stream);

/* dat_plan_test_stall -- TEST HOOK for the bounded wait of dat_step: sets the plan's wait limit to
 * `wait_cycles` SM clock cycles (0 restores the default) and, if `layer` >= 0, marks that layer's norm
 * as never completing for the next call (its tile counter is pre-set on the host side of the stream so
 * that the count cannot be reached): work items that need the layer give up after the limit and the
 * call ends with DAT_STATUS_TIMEOUT.  Nothing else uses this.  Errors: ARG, CUDA. */
int dat_plan_test_stall(dat_plan_t *plan, int64_t wait_cycles, int64_t layer, void *stream);

/* dat_step_host -- dat_step for callers whose data lives in HOST memory: copies theta, mom and
 * the M gradient buffers to plan-owned device staging buffers, runs dat_step, copies theta and
 * mom back, and synchronises `stream` before returning.
 *   theta_host, mom_host   host fp32[d], updated in place (pinned memory makes the copies fast).
 *   grads_host             host array of M host pointers, fp32[d] each.
 * The first call allocates the staging buffers ((M+2)*d*4 bytes, kept until the plan is
 * destroyed).  Errors: ARG, NOMEM, CUDA. */
int dat_step_host(dat_plan_t *plan, float *theta_host, float *mom_host,
                  const float *const *grads_host, uint64_t seed, uint64_t step,
                  const dat_hparams_t *hp, void *stream);

/* Synchronises `stream`, copies the plan's status word to *flags_out and clears it.  If the word carries
 * DAT_STATUS_TIMEOUT, the counters that the interrupted call left mid-way are cleared as well. */
int dat_get_status(dat_plan_t *plan, uint32_t *flags_out, void *stream);

/* Number of kernels the library has launched for this plan since it was created. */
int64_t dat_plan_launch_count(const dat_plan_t *plan);

/* Text for a DAT_ERR_* code (static storage). */
const char *dat_strerror(int code);

/* The cudaError_t value (as int) of the last failed CUDA call made for this plan, 0 if none. */
int dat_last_cuda_error(const dat_plan_t *plan);

#ifdef __cplusplus
}
#endif
#endif /* DAT_H_ */
