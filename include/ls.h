/*
 * ls.h -- C ABI of the local-update SGD library for one NVIDIA B200 (sm_100a).
 *
 * The library runs the data-parallel hot path of periodic-averaging SGD
 * (PASGD, Section 2 of "Adaptive Communication Strategies to Achieve the Best
 * Error-Runtime Trade-off in Local-Update SGD") for m model replicas that all
 * live in one GPU's memory, and the AdaComm communication-period rule
 * (Section 4.2).  Every arithmetic step runs in CUDA kernels of this library;
 * there is no CPU fallback.
 *
 * Conventions
 *  - Every function returns an int status: LS_OK (0) or a negative LS_ERR_*.
 *    Nothing throws or aborts across this boundary.  ls_strerror() names a code.
 *  - "dev" pointers are CUDA device pointers on the current device, "host"
 *    pointers are ordinary host memory.  The library allocates no device
 *    memory: the caller allocates one state block of ls_state_bytes() bytes
 *    (256-byte aligned) and lends it to the handle until ls_destroy().
 *  - Kernels are enqueued on the CUDA stream given to ls_create() and the call
 *    returns without waiting unless stated otherwise.  An asynchronous CUDA
 *    error surfaces as LS_ERR_CUDA from a later call or from ls_sync().
 *  - A handle is not thread-safe.
 *
 * Model: a fully connected network
 *      x -> W_L relu( ... relu(W_1 x + b_1) ... ) + b_L
 *  with dims = (d_in, h_1, ..., d_out).  n_layers == 1 is a linear model
 *  (softmax regression, or least squares with LS_LOSS_MSE_HALF and d_out == 1).
 *
 * Flat parameter layout of one replica (P = ls_param_count() floats): for
 *  l = 1..L the matrix W_l as [dims[l]][dims[l-1]] row-major, then b_l
 *  (dims[l] floats) when has_bias.  Momentum buffers use the same layout.
 *  Inside the state block replica i's vector starts at i * ls_param_stride()
 *  floats (the stride is P rounded up to a multiple of 64 floats).
 */
#ifndef LS_H_
#define LS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LS_MAX_LAYERS 8
#define LS_MAX_REPLICAS 64
#define LS_MAX_BATCH 1024
#define LS_MAX_OUT 1024          /* largest d_out (width of the loss layer) */

enum {
  LS_OK = 0,
  LS_ERR_INVALID_ARG = -1,       /* null pointer, size out of range, bad enum, non-finite number */
  LS_ERR_BAD_HANDLE = -2,
  LS_ERR_STATE_SIZE = -3,        /* state block too small or misaligned */
  LS_ERR_NO_DATASET = -4,        /* ls_bind_dataset() has not been called */
  LS_ERR_ROW_RANGE = -5,         /* a mini-batch would read past the bound dataset */
  LS_ERR_CUDA = -6,              /* a CUDA runtime call failed; ls_last_cuda_error() has its code */
  LS_ERR_UNSUPPORTED = -7,       /* valid request that the library does not implement (e.g. weight decay) */
  LS_ERR_OVERFLOW = -8,          /* a result does not fit its type */
  LS_ERR_DEVICE_TIMEOUT = -9,    /* a bounded wait inside a kernel ran out; results of that launch are invalid */
  LS_ERR_TOO_LARGE = -10,        /* a size exceeds a fixed capacity of the entry point */
  LS_ERR_EXCHANGE = -11          /* the exchange callback of ls_set_shard() reported a failure */
};

enum { LS_LOSS_SOFTMAX_CE = 0, LS_LOSS_MSE_HALF = 1 };
enum { LS_GEMM_FP32 = 0, LS_GEMM_BF16 = 1 };
/* What an averaging step does with the per-replica momentum buffers.
 * AVERAGE: replaced by their mean like the parameters (makes tau = 1 equal to
 *          synchronous momentum SGD on the m-fold batch).
 * KEEP:    left alone (the independent-buffer scheme of Section 5.3).
 * RESET:   cleared (the local half of the block-momentum scheme, Section 5.3).
 * BLOCK:   block momentum (Section 5.3): local buffers cleared, and the averaging step
 *          applies a global momentum buffer u to the period's accumulated step:
 *            u_j = beta_glob u_{j-1} + G_j,   x_{(j+1)tau+1} = x_{j tau+1} - eta u_j,
 *          with x_{j tau+1} the synchronized model the period started from and
 *          G_j = (x_{j tau+1} - mean_i x^(i)) / eta the averaged displacement in gradient units
 *          (the sum of the averaged gradients when the local steps are plain SGD).
 *          beta_glob is spec.block_momentum; see ls_average for the exact arithmetic. */
enum { LS_MOMENTUM_AVERAGE = 0, LS_MOMENTUM_KEEP = 1, LS_MOMENTUM_RESET = 2, LS_MOMENTUM_BLOCK = 3 };

typedef struct ls_model_spec {
  int32_t n_layers;                  /* L, 1..LS_MAX_LAYERS */
  int32_t dims[LS_MAX_LAYERS + 1];   /* dims[0..L] */
  int32_t loss;                      /* LS_LOSS_* */
  int32_t has_bias;                  /* 0 or 1 */
  int32_t gemm_dtype;                /* LS_GEMM_*: input type of the matrix products (accumulation is fp32) */
  int32_t momentum_mode;             /* LS_MOMENTUM_* */
  float weight_decay;                /* must be 0 */
  float block_momentum;              /* beta_glob of Section 5.3, 0 <= beta < 1; read only in LS_MOMENTUM_BLOCK */
} ls_model_spec;

typedef struct ls_handle ls_handle;

const char* ls_strerror(int code);

/* ---- sizes ------------------------------------------------------------- */

/* P, the number of parameters of one replica.  (x in R^d of Section 2.) */
int ls_param_count(const ls_model_spec* spec, int64_t* P);

/* Housekeeping (no passage of the paper): bytes of the caller-allocated state block for m replicas and
 * mini-batches of `batch` rows: parameters, momentum, bf16 weight copies (bf16 models),
 * activation / gradient workspace, staging for host batches. */
int ls_state_bytes(int m, const ls_model_spec* spec, int batch, size_t* bytes);

/* ---- life cycle -------------------------------------------------------- */

/* Create a handle for m replicas (1..LS_MAX_REPLICAS) that train with
 * learning rate lr (eta of Section 2) and momentum factor `momentum`
 * (0 <= momentum < 1; 0 means plain SGD and the buffers are never touched).
 * state_dev: device block of >= ls_state_bytes() bytes, 256-byte aligned; it is
 * borrowed until ls_destroy().  All parameters and momentum buffers start at
 * zero (enqueued on `cuda_stream`, a cudaStream_t passed as void*, may be 0).
 * Creates one auxiliary CUDA stream and a few events; allocates a small pinned
 * host buffer; no device memory. */
int ls_create(ls_handle** h, int m, const ls_model_spec* spec, float lr, float momentum, int batch,
              void* state_dev, size_t state_bytes, void* cuda_stream);
int ls_destroy(ls_handle* h);
/* Wait for everything enqueued so far; returns LS_ERR_CUDA if any of it failed.
 * Every wait inside the kernels (on a barrier, on a copy) is bounded; one that runs out makes its kernel
 * record a code in the state block and return.  ls_sync() and every call that waits for the stream itself
 * (ls_eval_loss, ls_local_steps_host, the decision points of ls_run / ls_run_refined / ls_run_timed, the state
 * accessors) then return LS_ERR_DEVICE_TIMEOUT once and clear the record: the results of the launches since the
 * last successful wait are invalid (restore the replicas with ls_set_state), the handle itself stays usable. */
int ls_sync(ls_handle* h);
/* Housekeeping (no passage of the paper): exercises the report path above without touching any other kernel.
 * Enqueues a one-thread kernel that waits, for at most limit_cycles SM clock ticks (1 .. 2e9), on a barrier on
 * which nothing ever arrives, gives up, and records the failure like a training kernel would.  The next
 * ls_sync() returns LS_ERR_DEVICE_TIMEOUT, the one after it LS_OK.  Nothing faults or hangs: the wait is the
 * bounded one the library uses everywhere. */
int ls_selftest_wait_timeout(ls_handle* h, int64_t limit_cycles);
int ls_last_cuda_error(const ls_handle* h);
int ls_set_lr(ls_handle* h, float lr);

/* ---- replica state  (X_k = [x^(1) ... x^(m)] of the proof's notation) --- */

/* All workers start at the same point x_1 (Section 2): copy the P host floats
 * to every replica, clear every momentum buffer.  Synchronous. */
int ls_set_params(ls_handle* h, const float* x1_host);
/* Overwrite / read one replica's parameters and momentum (P host floats each;
 * either pointer may be NULL to skip it).  Synchronous. */
int ls_set_state(ls_handle* h, int replica, const float* params_host, const float* momentum_host);
int ls_get_state(ls_handle* h, int replica, float* params_host, float* momentum_host);
/* Device views of the packed replicas: base pointers and the stride between
 * replicas in floats.  The memory belongs to the state block. */
int ls_state_view(ls_handle* h, float** params_dev, float** momentum_dev, int64_t* stride_floats);

/* ---- data -------------------------------------------------------------- */

/* Housekeeping (the paper's workers read their partition of the training set, Section 5.1; here it is one
 * resident array).  Bind the training set resident in device memory: x_dev is [n_rows][dims[0]]
 * row-major, float for LS_GEMM_FP32 and bf16 for LS_GEMM_BF16 (16-byte aligned);
 * y_dev is int32[n_rows] class labels for LS_LOSS_SOFTMAX_CE (each in
 * [0, d_out)) or float[n_rows] targets for LS_LOSS_MSE_HALF.  Borrowed: must
 * stay valid while the handle uses it. */
int ls_bind_dataset(ls_handle* h, const void* x_dev, const void* y_dev, int64_t n_rows);

/* ---- the hot path ------------------------------------------------------ */

/* tau local updates on every replica, no communication (Section 2, PASGD
 * update rule, the case k mod tau != 0, applied tau times):
 *      for s = 0..tau-1, for every replica i independently:
 *          xi  = dataset rows [row_offset[s*m + i], + batch)
 *          g   = (1/|xi|) sum_{s in xi} grad f(x^(i); s)      (Section 2)
 *          v^(i) <- momentum * v^(i) + g ;  x^(i) <- x^(i) - lr * v^(i)
 * row_offset_host: host int64[tau][m], read before the call returns.
 * loss_dev: optional device float[tau][m]; entry [s][i] receives the mean loss
 * of replica i's mini-batch at step s, evaluated before that step's update.
 * Errors: tau < 1, NULL offsets, a batch outside the dataset. */
int ls_local_steps(ls_handle* h, int tau, const int64_t* row_offset_host, float* loss_dev);

/* One whole communication period: the tau local steps of ls_local_steps followed by
 * the averaging step of ls_average (Section 2, PASGD update rule: the update of
 * iteration k is averaged when k mod tau = 0), in one call.  The state after the
 * call is bit for bit the state after ls_local_steps(tau) then ls_average().
 * Arguments and errors as ls_local_steps. */
int ls_local_steps_avg(ls_handle* h, int tau, const int64_t* row_offset_host, float* loss_dev);

/* Same steps, but the mini-batches come from host memory and the losses go
 * back to host memory: x_host is [tau][m][batch][dims[0]] (float or bf16 as
 * for ls_bind_dataset), y_host [tau][m][batch] (int32 or float), loss_host
 * float[tau][m].  Pinned host memory lets the copies overlap the kernels of
 * the previous step.  Synchronous: returns when loss_host is filled. */
int ls_local_steps_host(ls_handle* h, int tau, const void* x_host, const void* y_host, float* loss_host);

/* Model averaging (Section 2, PASGD update rule, the case k mod tau = 0;
 * X <- X J with J = 1 1^T / m): every replica's parameters are replaced by the
 * mean over replicas; momentum buffers follow spec.momentum_mode.
 * The mean is defined to the bit: s = x^(0); s = s + x^(j) for j = 1..m-1 in
 * fp32, then one fp32 division by (float)m.  Afterwards all replicas are
 * bitwise equal.
 * LS_MOMENTUM_BLOCK: with `mean` as above, a the model the period started from
 * and u the global buffer (both kept in the state block, a = x_1 and u = 0 after
 * ls_set_params), in fp32 with every operation rounded on its own:
 *   d = a - mean;  G = d / lr;  u' = beta*u + G;  x' = a - lr*u'
 * x' replaces every replica's parameters and a, u' replaces u, the local
 * momentum buffers are cleared.  lr is the rate in force when ls_average runs. */
int ls_average(ls_handle* h);

/* ---- one job on several GPUs --------------------------------------------------
 * The paper's own layout (Section 2: m workers, models averaged "by a fusion node or by performing an
 * all-node broadcast"; its experiments ran one worker per GPU): the m_total replicas of a job are dealt out in
 * index order over n_gpus GPUs, one process and one handle per GPU, m = m_total / n_gpus replicas in each
 * handle.  Local steps need no communication.  The averaging step becomes
 *     p_g   = x^(0) + x^(1) + ... + x^(m-1)            on GPU g, over its own replicas in index order, fp32
 *     total = p_0 + p_1 + ... + p_{n_gpus-1}           in rank order, fp32, after ONE exchange that brings every
 *                                                      GPU's partial sum into this GPU's own memory
 *     mean  = total / (float)m_total                   written to every local replica
 * (the same for the momentum buffers in LS_MOMENTUM_AVERAGE).  This GROUPED order replaces the sequential
 * order of ls_average() on such a handle: it rounds differently for 1 < n_gpus < m_total, is identical for
 * n_gpus = 1, is fixed, and gives every GPU the same bits, so all m_total replicas end bitwise equal.
 * LS_MOMENTUM_BLOCK is not available on several GPUs (LS_ERR_UNSUPPORTED).
 *
 * The library links no communication library and never reads another GPU's memory: the exchange is the
 * caller's (an all-gather, e.g. NCCL through torch.distributed), handed over as a callback. */

/* exchange(ctx, partial_dev, gathered_dev, bytes, n_gpus): gathered_dev[g*bytes .. (g+1)*bytes) must receive
 * rank g's `bytes` bytes at partial_dev, for every g (this rank's own included).  The copy must be ordered
 * after the work already enqueued on the handle's stream and before anything enqueued on it afterwards
 * (enqueue the collective on that stream, or make the stream wait for it).  Returns 0 on success. */
typedef int (*ls_exchange_fn)(void* ctx, const float* partial_dev, float* gathered_dev, size_t bytes, int n_gpus);

/* Floats that partial_dev of ls_set_shard() must hold (two padded replica vectors: parameters and momentum);
 * gathered_dev holds n_gpus times as many. */
int ls_shard_buffer_floats(const ls_handle* h, int64_t* floats);

/* Declare that this handle's m replicas are rank-local shares of a job of m_total = n_gpus * m replicas.  From
 * then on every averaging step of the handle (ls_average, ls_local_steps_avg, the run loops) is the grouped
 * average above, with one call of `exchange` per averaging step.  partial_dev / gathered_dev: caller-allocated
 * device buffers (256-byte aligned, sizes above), borrowed until ls_destroy() or ls_set_shard(h, 0, ...).
 * n_gpus = 1 needs no callback (and equals ls_average() bit for bit); n_gpus = 0 switches back.
 * All ranks must call the hot-path functions in the same order (the exchange is collective); the controller
 * needs no exchange of its own: every rank evaluates the same synchronized model on the same probe rows and
 * reaches the same decision. */
int ls_set_shard(ls_handle* h, int n_gpus, int m_total, float* partial_dev, float* gathered_dev, ls_exchange_fn exchange,
                 void* ctx);

/* The two halves of the grouped average for callers that run the exchange themselves: the partial sums of this
 * handle's replicas into partial_dev, and, given all ranks' partial sums in rank order, the mean into every
 * local replica (momentum buffers as in ls_average). */
int ls_shard_partial_sum(ls_handle* h, float* partial_dev);
int ls_shard_average(ls_handle* h, const float* gathered_dev, int n_gpus, int m_total);

/* The same two kernels on raw buffers (32-byte aligned, strides multiples of 8 floats):
 * out_dev[0..P) = sum of the m vectors at buf_dev + j*stride in index order;
 * every one of the m_local vectors at dst_dev + j*dst_stride = (sum of the G vectors at
 * partials_dev + g*part_stride, in that order) / (float)m_total. */
int ls_partial_sum_flat(const float* buf_dev, int m, int64_t P, int64_t stride, float* out_dev, void* cuda_stream);
int ls_combine_partials_flat(const float* partials_dev, int G, int64_t part_stride, int m_total, int64_t P,
                             float* dst_dev, int m_local, int64_t dst_stride, void* cuda_stream);

/* Block-momentum state of a LS_MOMENTUM_BLOCK handle in the flat interface layout
 * (P floats each): the period-start model and the global buffer.  Either pointer
 * may be NULL.  Host memory; synchronous.  LS_ERR_UNSUPPORTED in other modes. */
int ls_set_block_state(ls_handle* h, const float* anchor_host, const float* u_host);
int ls_get_block_state(ls_handle* h, float* anchor_host, float* u_host);

/* The block-momentum averaging kernel on raw buffers: buf_dev as for
 * ls_average_flat, anchor_dev and u_dev vectors of P floats (device), lr > 0,
 * beta >= 0.  Same arithmetic as ls_average in LS_MOMENTUM_BLOCK. */
int ls_block_average_flat(float* buf_dev, float* anchor_dev, float* u_dev, int m, int64_t P, int64_t stride,
                          float lr, float beta, void* cuda_stream);

/* The averaging kernel on a raw buffer: m vectors of P floats, vector j
 * starting at buf_dev + j*stride floats (stride >= P).  Same arithmetic as
 * ls_average().  Fastest when buf_dev is 32-byte aligned and stride is a
 * multiple of 8 floats (256-bit accesses); 16-byte alignment and a stride
 * multiple of 4 give 128-bit accesses; anything else runs element by element. */
int ls_average_flat(float* buf_dev, int m, int64_t P, int64_t stride, void* cuda_stream);

/* Training loss of one replica on dataset rows [row_offset, +n_rows), the
 * empirical risk F of Section 2 restricted to those rows; n_rows must be a
 * positive multiple of `batch`.  Forward pass only.  Synchronous; writes one
 * host float. */
int ls_eval_loss(ls_handle* h, int replica, int64_t row_offset, int64_t n_rows, float* F_host);

/* AdaComm basic update rule (Section 4.2):
 *      tau_l = ceil( sqrt(F_t / F_0) * tau_0 ),   F_inf taken as 0,
 * evaluated in IEEE double exactly as written, clamped below at 1 (growth
 * above tau_0 is allowed).  Pure host function.  Returns the new period (>= 1)
 * or a negative LS_ERR_* (F_0 <= 0, F_t < 0, non-finite input, tau_0 < 1,
 * result beyond INT32_MAX). */
int adacomm_next_tau(double F_t, double F_0, int tau_0);

/* AdaComm with the refinements of Section 4.3:
 *   candidate (Section 4.3.2, learning-rate coupling)   c = ceil( sqrt( (lr_0/lr_l) * F_t/F_0 ) * tau_0 ), >= 1
 *   faster decay when training saturates (Section 4.3.1, slack s):
 *        tau_l = c  if c + slack < tau_prev,  else ceil(gamma * tau_prev), >= 1
 *   lr_changed != 0 (first decision after the learning rate changed): c is returned as it is, so the period
 *   may grow when the rate drops.
 * Pure host function, IEEE double.  Returns the period or a negative LS_ERR_* (non-finite input, F_0 <= 0,
 * F_t < 0, tau_0 < 1, tau_prev < 1, gamma outside (0, 1], slack < 0, a learning rate <= 0). */
int adacomm_next_tau_refined(double F_t, double F_0, int tau_0, int tau_prev, double gamma, int slack, double lr_0,
                             double lr_l, int lr_changed);

/* Options of ls_run_refined(). */
typedef struct ls_adacomm_opts {
  double gamma;              /* decay factor of Section 4.3.1, in (0, 1]; the paper uses 1/2 */
  int32_t slack;             /* slack variable s of Section 4.3.1, >= 0 */
  int32_t n_decay;           /* number of scheduled learning-rate decays */
  const int64_t* decay_at;   /* host, ascending: iteration counts at which a decay is scheduled */
  double decay_factor;       /* lr <- lr * decay_factor (the paper divides by 10) */
} ls_adacomm_opts;

/* ls_run() with the refined rules: the period is chosen by adacomm_next_tau_refined(), and a scheduled
 * learning-rate decay is applied at the first decision point at or past its iteration at which the period in
 * force is 1 (Section 4.3.2: let the period decay to 1 first); one decay per decision.  interval must be >= 1.
 * The handle's learning rate is changed by the decays (read it back with ls_get_lr()). */
int ls_run_refined(ls_handle* h, int64_t K, int tau_0, int interval, int64_t probe_rows,
                   const int64_t* row_offset_host, float* loss_dev, const ls_adacomm_opts* opts, int32_t* period_tau,
                   int64_t max_periods, int64_t* n_periods, int64_t* decision_k, float* decision_F,
                   int32_t* decision_tau, int64_t max_decisions, int64_t* n_decisions, float* F0_host);
int ls_get_lr(const ls_handle* h, float* lr);

/* Whole training run in native code: K local iterations cut into periods of
 * tau local steps, each followed by ls_average().  With interval > 0 the
 * period is re-chosen by adacomm_next_tau() at the first averaging point at or
 * past each multiple of `interval` iterations, from the loss of replica 0 on
 * dataset rows [0, probe_rows) (F_0 is that loss at the starting point);
 * interval == 0 keeps tau fixed.  A period is never cut by an interval
 * boundary; the last period is cut at K and averaged.
 * row_offset_host: int64[K][m].  loss_dev: optional device float[K][m].
 * Outputs (host, optional): period_tau[max_periods] / n_periods list the period
 * lengths requested; decision_k / decision_F / decision_tau [max_decisions] /
 * n_decisions log every AdaComm decision; F0_host the initial loss. */
int ls_run(ls_handle* h, int64_t K, int tau_0, int interval, int64_t probe_rows,
           const int64_t* row_offset_host, float* loss_dev,
           int32_t* period_tau, int64_t max_periods, int64_t* n_periods,
           int64_t* decision_k, float* decision_F, int32_t* decision_tau, int64_t max_decisions,
           int64_t* n_decisions, float* F0_host);

/* The same run with the intervals of Section 4 as the paper defines them: training is cut into
 * wall-clock intervals of length T0_ms, and the period is re-chosen at the first averaging point
 * after each interval boundary (the clock is the host's steady clock, read after the stream has
 * drained at every averaging point, starting when the first local step is enqueued).  The schedule
 * depends on how fast the machine is, so it is not reproducible; what is reproducible is that every
 * logged decision equals adacomm_next_tau(decision_F, F_0, tau_0).  T0_ms <= 0 decides at every
 * averaging point.  decision_ms (optional, [max_decisions]) receives the elapsed time of each decision. */
int ls_run_timed(ls_handle* h, int64_t K, int tau_0, double T0_ms, int64_t probe_rows,
                 const int64_t* row_offset_host, float* loss_dev,
                 int32_t* period_tau, int64_t max_periods, int64_t* n_periods,
                 int64_t* decision_k, float* decision_F, int32_t* decision_tau, double* decision_ms,
                 int64_t max_decisions, int64_t* n_decisions, float* F0_host);

/* ---- runtime model (host only; Sections 2-4) -------------------------------
 * The delay model and the runtime / error-runtime formulas that motivate the choice of the period.
 * Pure host functions: no GPU, no handle. */
enum { LS_DELAY_CONSTANT = 0, LS_DELAY_LOG2 = 1, LS_DELAY_TREE = 2, LS_DELAY_LINEAR = 3 };
/* D = D0 * s(m) with s(m) = 1, log2 m, 2 log2 m (reduction tree) or m  (Section 2, delay model). */
int ls_delay(double D0, int m, int scaling, double* D);
/* E[T_sync] / E[T_P-Avg] = (1 + alpha) / (1 + alpha / tau) for constant Y and D, alpha = D / Y (Section 3.2). */
int ls_speedup(double alpha, int tau, double* speedup);
/* Theorem 1: 2 (F1 - Finf) / (lr T) (Y + D / tau) + lr L sigma2 / m + lr^2 L^2 sigma2 (tau - 1). */
int ls_error_bound(double T, double F1, double Finf, double lr, double L, double sigma2, int m, int tau, double Y,
                   double D, double* bound);
/* Theorem 2: tau* = sqrt(2 (F1 - Finf) D / (lr^3 L^2 sigma2 T)). */
int ls_tau_star(double F1, double Finf, double D, double lr, double L, double sigma2, double T, double* tau);
/* Monte-Carlo means of the runtime per iteration (Section 3.1) over n_periods periods of tau local
 * steps of m workers: t_sync_mean of T_sync = max_i Y_i + D (every local step followed by a
 * broadcast), t_pavg_mean of T_P-Avg = max_i (sum_k Y_ik / tau) + D / tau, on the same draws.
 * Y_ik is exponential with mean y_mean (exponential != 0) or the constant y_mean.  The draw of
 * (period p, step k, worker i) is -y_mean ln((x + 0.5) / 2^32), x the first word of
 * Philox4x32-10(counter = (p lo, p hi, k, i), key = (seed lo, seed hi)). */
int ls_simulate_runtime(int m, int tau, int64_t n_periods, double y_mean, double D, uint64_t seed, int exponential,
                        double* t_sync_mean, double* t_pavg_mean);
/* One block of Philox4x32-10 (Salmon et al., SC'11). */
int ls_philox4x32_10(const uint32_t counter[4], const uint32_t key[2], uint32_t out[4]);

/* Mean loss of a linear model on device-resident rows, for callers that must not allocate.
 * (The paper has no counterpart: this entry point exists for deployment reasons only.)
 *
 * Some callers cannot obtain device memory when they need a loss value: code that runs inside a
 * memory pool owned by somebody else, a monitoring hook that fires when the device is nearly
 * full, a plugin that is forbidden to call cudaMalloc, code that must not disturb an allocator's
 * fragmentation state.  ls_eval_loss() needs the caller to have allocated a whole state block,
 * because the output-layer kernel keeps per-row losses, CTA counters and chunk offsets in
 * scratch memory.  Here that scratch is a fixed array inside the library image (about 260 KB of
 * every GPU that loads the library, held until the process exits), and the call allocates
 * nothing: no cudaMalloc, no cudaFree, no allocating library routine.
 *
 * Computes, for chunk c = 0 .. n_rows/chunk_rows - 1 of chunk_rows consecutive rows, the mean
 * loss of z = W x + b on those rows and writes it to chunk_loss_dev[c] (the caller's own device
 * buffer).  W_dev is float [d_out][d_in], bias_dev float [d_out] or NULL, x_dev float
 * [n_rows][d_in] (16-byte aligned for the fast path), y_dev int32 labels (LS_LOSS_SOFTMAX_CE) or
 * float targets (LS_LOSS_MSE_HALF, d_out == 1).  Same kernel and arithmetic as ls_eval_loss() on a
 * one-layer fp32 model with mini-batch chunk_rows.  Enqueued on cuda_stream; returns at once.
 *
 * Limits: d_out <= 16, at most 256 chunks and 65 536 rows per call, chunk_rows <= LS_MAX_BATCH;
 * beyond them the call returns LS_ERR_TOO_LARGE and does nothing.
 * The first call on each device looks up the scratch array's device address (with that device
 * current); make that first call outside any stream capture.
 * All calls on a device share the one scratch array: it keeps the previous call's contents (the
 * entry point re-clears what must start at zero), and two calls whose kernels overlap on the GPU
 * (different streams) race on it -- serialise them. */
int ls_linear_loss_static(const float* W_dev, const float* bias_dev, const float* x_dev, const void* y_dev,
                          int64_t n_rows, int d_in, int d_out, int loss, int chunk_rows, float* chunk_loss_dev,
                          void* cuda_stream);

/* Per-kernel device timing.  Between ls_profile_begin() and ls_profile_end()
 * every launch of a kernel class selected by class_mask (bit c = class c; for
 * the per-layer classes only layer `layer`, 0-based, or all layers when
 * layer < 0) is bracketed by a pair of CUDA events on the handle's stream.
 * ls_profile_end() waits for the stream and adds up, per class and layer, the
 * elapsed milliseconds and the number of launches into
 * ms[LS_K_CLASSES * LS_MAX_LAYERS] and launches[...] (index class*LS_MAX_LAYERS
 * + layer; LS_K_LOSS uses layer 0; LS_K_AVG uses layer 0 for the averaging
 * kernel and layer 1 for the launch that does the last weight update of a
 * period and its averaging step together, both whatever `layer` says).  At most
 * 16384 launches are recorded per profile; later ones are run but not timed. */
enum { LS_K_FWD = 0, LS_K_LOSS = 1, LS_K_DX = 2, LS_K_DW = 3, LS_K_BIAS = 4, LS_K_AVG = 5, LS_K_CLASSES = 6 };
int ls_profile_begin(ls_handle* h, uint32_t class_mask, int layer);
int ls_profile_end(ls_handle* h, double* ms, int64_t* launches);

/* Number of kernels this handle has launched so far. */
int ls_launch_count(const ls_handle* h, int64_t* n);

#ifdef __cplusplus
}
#endif
#endif /* LS_H_ */
