/*
 * sgdb.h -- C ABI of libsgdb: the synchronous parameter-server step with backup
 * workers ("first N of N+b"), for one NVIDIA B200 (sm_100a).
 *
 * Source of the operations: "Revisiting Distributed Synchronous SGD"
 * (arXiv 1604.00981), Section 3 (backup workers) and Algorithm 4 (Sync-SGD
 * parameter server): for iteration t the server keeps gradients whose tag equals
 * t, stops at the N-th such arrival, drops everything else, and updates the
 * parameters with the mean of the kept N.
 *
 * Notation (the paper's): N workers whose gradients are used, b backup workers,
 * W = N + b rows, t the server's iteration, theta the parameters, G the
 * gradients.  Workers are numbered 0..W-1 here (the paper counts from 1).
 *
 * Conventions shared by every call unless its comment says otherwise
 *   - `d_` pointers are DEVICE memory and `h_` pointers HOST memory, both owned by
 *     the caller; the library never frees or keeps them.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls only enqueue work; they never synchronise the stream, except the
 *     `_host` entry point, which says so.
 *   - Nothing is allocated by the library; the only memory it touches is what the
 *     caller passes -- except sgdb_step_host_static, which works in a fixed array that is
 *     part of the library image.
 *   - Arguments that can be checked on the host (null pointers, N < 1, b < 0,
 *     N + b > SGDB_MAX_WORKERS, P < 0, ld < P, misaligned base pointers, unknown
 *     enum values, non-finite hyper-parameters) make the call return
 *     SGDB_ERR_INVALID_ARG (or SGDB_ERR_UNSUPPORTED) without launching anything.
 *   - Conditions only the device can see land in a caller-owned device word
 *     (`d_info`); when that word says SGDB_ERR_INSUFFICIENT, theta, optimizer
 *     state and mean are left bit-for-bit untouched (Algorithm 4 does not update
 *     before N current gradients exist).
 *   - The gradient matrix G is row-major, row w = worker w, `ld` elements between
 *     row starts (ld >= P), element type sgdb_dtype_t.  theta, optimizer state,
 *     mean and accumulator are fp32.
 *   - Base pointers of G, theta, state, mean and acc must be 16-byte aligned in
 *     the flat calls.  Rows are streamed with 16-byte bulk copies when
 *     ld * sizeof(element) is a multiple of 16; any other ld is accepted and
 *     takes an element-wise load path with identical results.  On the 16-byte path
 *     the padding columns of a kept row up to the next 16-byte boundary after its last
 *     used column may be read; their values are never used.
 *   - Pass the server's real iteration number t and let it grow by one per iteration, as
 *     Algorithm 4 does: the fused calls walk through the columns forward when t is even and
 *     backward when t is odd, so that an iteration starts with the parameters and state the
 *     previous one wrote last and finds them in cache.  Results do not depend on it; a constant
 *     t only forgoes that gain (about 1-2 % of the step).
 *   - Summation order is fixed: the kept rows are added one after another in
 *     arrival order, starting from +0, in fp32, and the sum is divided by N once.
 *     Results are therefore bit-reproducible run to run and identical between
 *     the fused, the separate and the accumulate-on-arrival calls.
 */
#ifndef SGDB_H_
#define SGDB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SGDB_MAX_WORKERS 1024  /* largest accepted W = N + b */
#define SGDB_MAX_SEGMENTS 4096 /* largest accepted segment-table length */

typedef enum {
  SGDB_OK = 0,
  SGDB_ERR_INVALID_ARG = 1,
  SGDB_ERR_INSUFFICIENT = 2, /* fewer than N workers with tag == t and a finite arrival */
  SGDB_ERR_CUDA = 3,         /* a CUDA runtime call or a launch failed */
  SGDB_ERR_UNSUPPORTED = 4,
  SGDB_ERR_TIMEOUT = 5       /* a bounded on-chip wait ran out (never expected) */
} sgdb_status_t;

typedef enum { SGDB_F32 = 0, SGDB_BF16 = 1 } sgdb_dtype_t; /* storage type of G's rows */

typedef enum {
  SGDB_SGD = 0,      /* theta -= lr * g                                   (Section 1.1, SGD rule)      */
  SGDB_MOMENTUM = 1, /* v = momentum*v + g;  theta -= lr * v                                           */
  SGDB_RMSPROP = 2,  /* s = decay*s + (1-decay)*g^2;  m = momentum*m + lr*g/sqrt(s+eps);  theta -= m   */
  SGDB_ADAM = 3,     /* m = beta1*m + (1-beta1)*g;  v = beta2*v + (1-beta2)*g^2;
                        theta -= lr * (m/(1-beta1^step)) / (sqrt(v/(1-beta2^step)) + eps)             */
  SGDB_ADAGRAD = 4   /* s = s + g^2;  theta -= lr * g / (sqrt(s) + eps)                               */
} sgdb_opt_kind_t;

/*
 * Optimizer rule and hyper-parameters, passed by pointer from HOST memory and
 * read during the call.  g is the mean of the N kept gradients; `lr` multiplies
 * that mean (Algorithm 4 writes gamma_t / N times the sum).  The paper names the
 * family (Section 1.1) and uses RMSProp with momentum in its experiments
 * (Appendix A) without printing equations; the forms above are the ones this
 * library computes.  state0/state1 per rule: SGD none; MOMENTUM v/-; RMSPROP
 * s/m; ADAM m/v; ADAGRAD s/-.  `step` is the 1-based count of updates including this one and
 * matters to ADAM only.
 */
typedef struct sgdb_opt {
  int32_t kind; /* sgdb_opt_kind_t */
  float lr;
  float momentum;
  float decay;
  float beta1;
  float beta2;
  float eps;
  int64_t step;
} sgdb_opt_t;

/*
 * One tensor of a multi-tensor model (the paper's parameter server updates the
 * model variable by variable; Section 3.1 follows "one variable", Appendix A.3
 * sends layers separately).  All pointers are device pointers; only element
 * alignment (4 bytes, 2 for bf16 gradients) is required, 16-byte alignment of
 * every pointer and of ld * sizeof(element) selects the fast path per segment.
 */
typedef struct sgdb_segment {
  void *theta;      /* fp32 [len] */
  void *state0;     /* fp32 [len] or NULL when the rule has no first state  */
  void *state1;     /* fp32 [len] or NULL when the rule has no second state */
  const void *grad; /* [W x ld], this tensor's gradient rows, one per worker */
  int64_t ld;       /* elements between row starts, >= len */
  int64_t len;      /* elements in this tensor, >= 0 */
} sgdb_segment_t;

/*
 * sgdb_select -- which gradients the server uses at iteration t.
 * Section 3 (the first N to arrive are used, the slowest b are dropped) and
 * Algorithm 4 (a gradient counts only if its tag equals t).
 *
 *   d_arrival [W] fp32   arrival time of worker w's gradient; NaN or +-inf = never arrives
 *   d_tags    [W] int32  iteration the gradient was computed for
 *   t, N, b              server iteration, gradients to aggregate, backup workers; W = N + b
 *   d_mask    [W] uint8  out: 1 for the N kept workers, else 0
 *   d_order   [N] int32  out: kept worker ids in arrival sequence; equal arrival
 *                        times are ordered by lower worker id
 *   d_info    [2] int32  out: {number of valid workers, SGDB_OK or SGDB_ERR_INSUFFICIENT}
 *
 * When fewer than N workers are valid, d_mask and d_order are left untouched.
 */
sgdb_status_t sgdb_select(const float *d_arrival, const int32_t *d_tags, int32_t t, int32_t N,
                          int32_t b, uint8_t *d_mask, int32_t *d_order, int32_t *d_info,
                          void *stream);

/*
 * sgdb_aggregate -- mean of the kept gradients: (1/N) * sum over the kept G
 * (the sum in Algorithm 4's update line, before the learning rate).
 *
 *   d_grad  [W x ld] rows of type dt;  P columns used;  d_order [N] from sgdb_select
 *   d_info  [2] or NULL: when given and d_info[1] != SGDB_OK the kernel writes nothing
 *   d_mean  [P] fp32 out
 * Rows not named in d_order are never read.
 */
sgdb_status_t sgdb_aggregate(const void *d_grad, sgdb_dtype_t dt, int64_t P, int64_t ld, int32_t N,
                             const int32_t *d_order, const int32_t *d_info, float *d_mean,
                             void *stream);

/*
 * sgdb_update -- apply the optimizer rule to theta with a given mean gradient
 * (Algorithm 4's update line; Section 1.1 for the family of rules).
 *
 *   d_theta [P] in/out;  d_state0, d_state1 [P] in/out or NULL as the rule needs
 *   d_mean  [P] in;  opt: host pointer;  d_info as in sgdb_aggregate
 */
sgdb_status_t sgdb_update(float *d_theta, float *d_state0, float *d_state1, const float *d_mean,
                          int64_t P, const sgdb_opt_t *opt, const int32_t *d_info, void *stream);

/*
 * sgdb_step -- one whole iteration of Algorithm 4's loop body: select,
 * aggregate and update, in a single kernel launch; the mean is never written to
 * memory.  Arguments as in the three calls above; d_mask, d_order and d_info are
 * outputs here.
 */
sgdb_status_t sgdb_step(const void *d_grad, sgdb_dtype_t dt, int64_t P, int64_t ld,
                        const float *d_arrival, const int32_t *d_tags, int32_t t, int32_t N,
                        int32_t b, float *d_theta, float *d_state0, float *d_state1,
                        const sgdb_opt_t *opt, uint8_t *d_mask, int32_t *d_order, int32_t *d_info,
                        void *stream);

/*
 * sgdb_step_ema -- sgdb_step plus the line that follows the update in Algorithm 4:
 * the exponential moving average of the parameters (Section 1.1),
 *     avg <- alpha * avg + (1 - alpha) * theta(t),
 * where theta(t) is the value of the parameters BEFORE this iteration's update, as
 * Algorithm 4 writes it.  Same launch, 8 more bytes per parameter.
 *   d_ema [P] fp32 in/out, 16-byte aligned.  The paper leaves the average before the
 *   first iteration undefined; initialise d_ema with theta(0), so that it equals
 *   theta(0) after iteration 0.  alpha in [0, 1] (the paper evaluates with 0.9999).
 * When fewer than N gradients are current, d_ema is untouched like everything else.
 */
sgdb_status_t sgdb_step_ema(const void *d_grad, sgdb_dtype_t dt, int64_t P, int64_t ld,
                            const float *d_arrival, const int32_t *d_tags, int32_t t, int32_t N,
                            int32_t b, float *d_theta, float *d_state0, float *d_state1,
                            const sgdb_opt_t *opt, float *d_ema, float alpha, uint8_t *d_mask,
                            int32_t *d_order, int32_t *d_info, void *stream);

/*
 * sgdb_ema -- the same average on its own, for callers of the separate calls
 * (Algorithm 4's last line): avg <- alpha * avg + (1 - alpha) * theta.  Call it
 * before sgdb_update to average the pre-update parameters as sgdb_step_ema does.
 * d_info as in sgdb_aggregate.
 */
sgdb_status_t sgdb_ema(float *d_ema, const float *d_theta, int64_t P, float alpha,
                       const int32_t *d_info, void *stream);

/*
 * sgdb_learning_rate -- the paper's learning-rate schedule (Appendix A.2, A.3), a host
 * computation: gamma0 * beta^(t*N / (2*T)), with T = |X| / B the number of mini-batches
 * in the data set.  N = number of aggregated workers for the synchronous rule; N = 1
 * gives the asynchronous rule gamma0 * beta^(t / (2*T)).  NaN for T <= 0, N < 1 or t < 0.
 */
double sgdb_learning_rate(double gamma0, double beta, int64_t t, int64_t N, double T);

/*
 * sgdb_select_deadline, sgdb_step_deadline -- the alternative the paper names in its
 * conclusion (Section 6): a time-out instead of backup workers.  The paper prints no
 * algorithm for it; this is Algorithm 4 with the stopping rule exchanged: the server
 * listens until `deadline`, keeps EVERY gradient tagged t that arrived by then
 * (arrival <= deadline, finite), drops the rest, and averages over the n it kept.
 *
 *   W            number of workers (rows of G, entries of d_arrival / d_tags / d_mask)
 *   deadline     fp32 seconds, +infinity = wait for everyone; NaN is refused
 *   n_min        1 <= n_min <= W: with fewer kept gradients the iteration does not
 *                complete (d_info[1] = SGDB_ERR_INSUFFICIENT, nothing else is touched)
 *   d_order [W]  out: the first n entries are the kept ids in arrival sequence
 *   d_info  [2]  out: {n, status}; the mean divides by n
 * sgdb_step_deadline is one launch, like sgdb_step.
 */
sgdb_status_t sgdb_select_deadline(const float *d_arrival, const int32_t *d_tags, int32_t t, int32_t W,
                                   float deadline, int32_t n_min, uint8_t *d_mask, int32_t *d_order,
                                   int32_t *d_info, void *stream);
sgdb_status_t sgdb_step_deadline(const void *d_grad, sgdb_dtype_t dt, int64_t P, int64_t ld,
                                 const float *d_arrival, const int32_t *d_tags, int32_t t, int32_t W,
                                 float deadline, int32_t n_min, float *d_theta, float *d_state0,
                                 float *d_state1, const sgdb_opt_t *opt, uint8_t *d_mask,
                                 int32_t *d_order, int32_t *d_info, void *stream);

/*
 * sgdb_step_segmented -- sgdb_step over a model stored as S separate tensors,
 * in one launch driven by a table in DEVICE memory (d_segments [S]).  One
 * selection serves all tensors, as one server iteration does in Algorithm 4.
 * S <= SGDB_MAX_SEGMENTS, otherwise SGDB_ERR_UNSUPPORTED.  The table cannot be
 * inspected from the host: a segment with a null theta or grad pointer, without a
 * state pointer its rule needs, with a pointer that is not aligned to its element type or
 * with ld < len is skipped by the kernel and d_info[1] then reads SGDB_ERR_INVALID_ARG (the
 * other segments are still updated).
 */
sgdb_status_t sgdb_step_segmented(const sgdb_segment_t *d_segments, int32_t S, sgdb_dtype_t dt,
                                  const float *d_arrival, const int32_t *d_tags, int32_t t,
                                  int32_t N, int32_t b, const sgdb_opt_t *opt, uint8_t *d_mask,
                                  int32_t *d_order, int32_t *d_info, void *stream);

/*
 * sgdb_step_segmented_ema -- sgdb_step_segmented that also keeps the parameter average of
 * Algorithm 4's last line (which the algorithm runs for every variable) for each tensor, in
 * the same launch, from the parameters as they were before the update (see sgdb_step_ema).
 *   d_ema [S]  DEVICE array of device pointers, entry i = fp32 [len_i] average of tensor i
 *              (element-aligned; 16-byte aligned is faster); a NULL entry: no average for
 *              that tensor.  alpha in [0, 1].
 *
 * sgdb_step_segmented_deadline -- sgdb_step_segmented with the time-out rule of
 * sgdb_step_deadline (Section 6): W workers, every gradient tagged t that arrived by
 * `deadline` is used, at least n_min of them; d_order has W entries, d_info = {n, status}.
 *
 * In all three calls an entry of the table whose pointers are missing or not aligned to
 * their element type, or whose ld is smaller than its len, is skipped and reported as
 * SGDB_ERR_INVALID_ARG in d_info[1].
 */
sgdb_status_t sgdb_step_segmented_ema(const sgdb_segment_t *d_segments, float *const *d_ema, float alpha,
                                      int32_t S, sgdb_dtype_t dt, const float *d_arrival,
                                      const int32_t *d_tags, int32_t t, int32_t N, int32_t b,
                                      const sgdb_opt_t *opt, uint8_t *d_mask, int32_t *d_order,
                                      int32_t *d_info, void *stream);
sgdb_status_t sgdb_step_segmented_deadline(const sgdb_segment_t *d_segments, int32_t S, sgdb_dtype_t dt,
                                           const float *d_arrival, const int32_t *d_tags, int32_t t,
                                           int32_t W, float deadline, int32_t n_min, const sgdb_opt_t *opt,
                                           uint8_t *d_mask, int32_t *d_order, int32_t *d_info,
                                           void *stream);

/*
 * sgdb_select_grouped, sgdb_step_grouped -- two-level aggregation: the gradients of workers
 * that share a machine are combined before they reach the server.  The paper names this in
 * its conclusion (Section 6) and prints no algorithm; here a machine takes a worker's place
 * in Algorithm 4 (Section 3 for the first-N rule):
 *   - worker w runs on machine d_group[w], 0 <= d_group[w] < M;
 *   - a machine's message is the mean of its workers' gradients and arrives when the
 *     slowest of them does (the maximum of their arrival times);
 *   - the message counts for iteration t only if every worker of the machine is tagged t
 *     and has a finite arrival time; a machine without workers sends nothing;
 *   - the server uses the first N messages to arrive (equal times: lower machine id) and
 *     moves theta by the mean of those N messages; rows of machines it drops are never read.
 *
 *   d_arrival, d_tags, d_group [W]   per worker;  W, M <= SGDB_MAX_WORKERS, 1 <= N <= M
 *   d_mask        [W] uint8  out: 1 for every worker whose gradient is used
 *   d_group_order [N] int32  out: the kept machines in the order their messages arrived
 *   d_order       [W] int32  out: the used workers in summation sequence -- machine by
 *                            machine in that order, within a machine by (arrival, id);
 *                            d_info[2] entries are written
 *   d_info        [3] int32  out: {machines whose message counts, status, workers used}
 * Summation: a machine's rows are added one after another from +0 and divided by their
 * number; the N messages are added one after another from +0 and divided by N (fp32).  The
 * result has the bits of sgdb_aggregate per machine followed by sgdb_step over the machines'
 * means.  With fewer than N messages that count, d_info[1] = SGDB_ERR_INSUFFICIENT and nothing
 * else is touched; a machine id outside [0, M) gives d_info[1] = SGDB_ERR_INVALID_ARG likewise.
 * sgdb_step_grouped is one launch.
 */
sgdb_status_t sgdb_select_grouped(const float *d_arrival, const int32_t *d_tags, const int32_t *d_group,
                                  int32_t t, int32_t W, int32_t M, int32_t N, uint8_t *d_mask,
                                  int32_t *d_group_order, int32_t *d_order, int32_t *d_info, void *stream);
sgdb_status_t sgdb_step_grouped(const void *d_grad, sgdb_dtype_t dt, int64_t P, int64_t ld,
                                const float *d_arrival, const int32_t *d_tags, const int32_t *d_group,
                                int32_t t, int32_t W, int32_t M, int32_t N, float *d_theta, float *d_state0,
                                float *d_state1, const sgdb_opt_t *opt, uint8_t *d_mask,
                                int32_t *d_group_order, int32_t *d_order, int32_t *d_info, void *stream);

/*
 * sgdb_step_rows, sgdb_step_rows_ordered, sgdb_shard_range -- the step as ONE of several
 * parameter servers runs it (Section 1.1: the parameters are split over servers, server j holds
 * theta[j], receives every worker's gradient of theta[j] and hands theta[j] back to the workers;
 * Algorithm 4 runs on every server; Algorithm 3 sends G[j] to server j and reads theta[j] from it).
 * This is the form for several GPUs: each GPU is server j for one range of columns, the workers'
 * gradients are whole rows that live in any GPU's memory, and every GPU keeps a full copy of theta
 * for its workers to read.
 *
 *   d_rows     [W] DEVICE array of device addresses: d_rows[w] = column `first` of worker w's
 *                  gradient, i.e. the first element server j is responsible for; `len` elements of
 *                  type dt are read from the kept rows, the others are never touched.  An address
 *                  may belong to this GPU or to a peer GPU whose memory is mapped into this process.
 *                  Element-aligned addresses are required; when every kept row is 16-byte aligned
 *                  the rows are pulled with bulk copies (never multicast), else with element loads,
 *                  same results.
 *   len            columns of this server's range (sgdb_shard_range gives ranges that keep every
 *                  server's addresses 16-byte aligned when the full rows are)
 *   d_theta, d_state0, d_state1 [len]  this server's range of the parameters and state, in/out,
 *                  this GPU's memory, 16-byte aligned
 *   d_replicas [R] DEVICE array of device addresses, R <= SGDB_MAX_REPLICAS, or NULL with R = 0:
 *                  d_replicas[r] = where copy r of this range lives (column `first` of a full copy
 *                  of theta, this GPU's memory or a peer's); the new parameters are stored to
 *                  d_theta and to every replica in the same pass (4 * R more bytes per column)
 *   selection      sgdb_step_rows takes it in the kernel's prologue like sgdb_step (d_arrival,
 *                  d_tags, t, N, b in; d_mask, d_order, d_info out): every server computes the same
 *                  selection from the same W numbers, so all ranges use the same N gradients.
 *                  sgdb_step_rows_ordered is given it: d_order [N] row ids in summation sequence
 *                  (each in [0, W)), d_info [2] in/out -- when d_info[1] != SGDB_OK on entry nothing
 *                  is done; the mean divides by N.
 * A null or misaligned address among the kept rows or the replicas, or a row id outside [0, W),
 * makes the kernel touch nothing and write SGDB_ERR_INVALID_ARG to d_info[1].
 * Summation order, arithmetic and therefore the bits of theta and state are those of sgdb_step on
 * the same columns.  One launch; no block waits for another GPU.  Ordering between GPUs is the
 * caller's: every kept gradient must be complete before the launch, and a replica may be read only
 * after the launches of all servers that write to it have completed (the barrier of the
 * synchronous protocol, Section 3).
 *
 * sgdb_step_rows_ordered also serves two-level aggregation across GPUs (Section 6, see
 * sgdb_step_grouped): each machine writes the mean of its workers' gradients (sgdb_select over its own
 * workers, then sgdb_aggregate), the servers then take the kept machines' means as rows, with
 * d_order = the d_group_order of sgdb_select_grouped; the result has the bits of sgdb_step_grouped.
 *
 * sgdb_shard_range (host computation): range j of n_servers over P columns, contiguous, in order,
 * together covering [0, P), every start a multiple of SGDB_SHARD_ALIGN columns; trailing ranges
 * may be empty.
 */
#define SGDB_MAX_REPLICAS 64 /* largest accepted R */
#define SGDB_SHARD_ALIGN 64  /* columns; keeps fp32 and bf16 rows 128-byte aligned at every range start */
sgdb_status_t sgdb_step_rows(const void *const *d_rows, sgdb_dtype_t dt, int64_t len,
                             const float *d_arrival, const int32_t *d_tags, int32_t t, int32_t N,
                             int32_t b, float *d_theta, float *d_state0, float *d_state1,
                             const sgdb_opt_t *opt, float *const *d_replicas, int32_t R,
                             uint8_t *d_mask, int32_t *d_order, int32_t *d_info, void *stream);
sgdb_status_t sgdb_step_rows_ordered(const void *const *d_rows, int32_t W, sgdb_dtype_t dt, int64_t len,
                                     int32_t N, const int32_t *d_order, int32_t *d_info, float *d_theta,
                                     float *d_state0, float *d_state1, const sgdb_opt_t *opt,
                                     float *const *d_replicas, int32_t R, void *stream);
sgdb_status_t sgdb_shard_range(int64_t P, int32_t n_servers, int32_t j, int64_t *first, int64_t *len);

/*
 * sgdb_enable_peer_access -- lets kernels launched on the CURRENT device read and write the memory of
 * `peer_device` (what sgdb_step_rows needs before it is given a peer's addresses; no counterpart in the
 * paper).  Enabling twice is fine; the current device itself is accepted and needs nothing.
 * SGDB_ERR_UNSUPPORTED when the two devices have no peer path, SGDB_ERR_INVALID_ARG for a device that does
 * not exist.  This is a one-time set-up call of the process, not part of an iteration.
 */
sgdb_status_t sgdb_enable_peer_access(int32_t peer_device);

/*
 * sgdb_accumulate_arrival -- Algorithm 4's inner loop taken literally: one
 * gradient per call, in the order the gradients reach the server.
 *
 *   d_row     [P] of type dt   the arriving gradient; any element-aligned address (a row of
 *                              a matrix with an odd pitch is fine; an address that is not a
 *                              multiple of the element size is refused), 16-byte aligned is faster
 *   row_tag, t                 its tag and the server's iteration
 *   d_acc     [P] fp32         running sum, owned by the caller; needs no clearing:
 *                              the first accepted arrival of an iteration overwrites it
 *   d_counter [4] int32        server state, zero-initialised once by the caller:
 *                              {accepted so far, arrivals seen, internal ticket,
 *                               lowest iteration still open}
 *   d_info    [2] int32 out    {0 dropped | 1 accumulated | 2 accumulated and updated,
 *                               accepted count after this call}
 * A row is accepted iff row_tag == t, t is still open and fewer than N rows have
 * been accepted; otherwise it is dropped and d_acc is not touched.  The N-th
 * accepted row triggers mean + optimizer update in the same launch, closes
 * iteration t and resets the accepted count.  Calls on one stream are ordered by
 * the stream; there are no device-side waits.  Calls for the same server state
 * must not overlap on the device.
 */
sgdb_status_t sgdb_accumulate_arrival(const void *d_row, sgdb_dtype_t dt, int32_t row_tag,
                                      int32_t t, int32_t N, int64_t P, float *d_acc,
                                      int32_t *d_counter, float *d_theta, float *d_state0,
                                      float *d_state1, const sgdb_opt_t *opt, int32_t *d_info,
                                      void *stream);

/*
 * sgdb_accumulate_arrival_ema -- sgdb_accumulate_arrival that also keeps the parameter
 * average of Algorithm 4's last line: d_ema [P] (fp32, 16-byte aligned) is updated as in
 * sgdb_step_ema, in the launch of the N-th accepted gradient and only then.
 */
sgdb_status_t sgdb_accumulate_arrival_ema(const void *d_row, sgdb_dtype_t dt, int32_t row_tag,
                                          int32_t t, int32_t N, int64_t P, float *d_acc,
                                          int32_t *d_counter, float *d_theta, float *d_state0,
                                          float *d_state1, const sgdb_opt_t *opt, float *d_ema,
                                          float alpha, int32_t *d_info, void *stream);

/*
 * sgdb_accumulate_arrival_deadline, sgdb_accumulate_close -- the time-out rule (Section 6, see
 * sgdb_select_deadline) with one gradient per call.  The server listens until `deadline`:
 * a gradient joins the running sum iff row_tag == t, iteration t is still open and
 * row_arrival is finite and <= deadline; there is no upper count.  d_info = {0 dropped |
 * 1 accumulated, gradients in the set after this call}.  d_row, d_acc, d_counter as in
 * sgdb_accumulate_arrival; row_arrival and deadline are host values (NaN deadline is refused).
 *
 * sgdb_accumulate_close says that the deadline of iteration t has passed.  With at least
 * n_min (>= 1) gradients in the set, theta moves by their mean (the divisor is the number
 * in the set), the set is emptied and iteration t + 1 opens: d_info = {2, that number}.
 * With fewer, or when t is already closed, nothing changes: d_info = {0, gradients in the
 * set}; the caller may keep delivering and close again later.  d_ema may be NULL; otherwise
 * the parameter average of Algorithm 4's last line moves with the update, as in sgdb_step_ema.
 * Delivered in arrival sequence, the result has the bits of sgdb_step_deadline.
 */
sgdb_status_t sgdb_accumulate_arrival_deadline(const void *d_row, sgdb_dtype_t dt, int32_t row_tag,
                                               float row_arrival, int32_t t, float deadline, int64_t P,
                                               float *d_acc, int32_t *d_counter, int32_t *d_info,
                                               void *stream);
sgdb_status_t sgdb_accumulate_close(int32_t t, int32_t n_min, int64_t P, const float *d_acc,
                                    int32_t *d_counter, float *d_theta, float *d_state0, float *d_state1,
                                    const sgdb_opt_t *opt, float *d_ema, float alpha, int32_t *d_info,
                                    void *stream);

/*
 * sgdb_step_host -- sgdb_step for a server whose gradients arrive in HOST memory
 * (the worker-to-server message of Algorithm 3 lands in host buffers) and whose
 * new parameters go back out to the workers (Algorithm 3 reads theta each
 * iteration).  theta and the optimizer state stay resident on the device.
 *
 *   h_grad [W x ld], h_arrival [W], h_tags [W]   host inputs (pinned memory makes
 *                                                the copies asynchronous and fast)
 *   d_theta, d_state0, d_state1                  device, in/out
 *   h_theta_out [P] or NULL                      host copy of the updated theta
 *   h_mask [W], h_order [N], h_info [2]          host outputs
 *   d_workspace, workspace_bytes                 device scratch owned by the caller, at
 *                                                least sgdb_step_host_workspace_bytes();
 *                                                16-byte aligned; contents undefined after
 * Only the N kept rows cross to the device.  The call synchronises `stream`
 * twice (after selection, and before returning) and returns the device-detected
 * status, e.g. SGDB_ERR_INSUFFICIENT, directly.
 */
sgdb_status_t sgdb_step_host(const void *h_grad, sgdb_dtype_t dt, int64_t P, int64_t ld,
                             const float *h_arrival, const int32_t *h_tags, int32_t t, int32_t N,
                             int32_t b, float *d_theta, float *d_state0, float *d_state1,
                             const sgdb_opt_t *opt, float *h_theta_out, uint8_t *h_mask,
                             int32_t *h_order, int32_t *h_info, void *d_workspace,
                             size_t workspace_bytes, void *stream);

/* Bytes of device workspace sgdb_step_host needs for these sizes (0 on invalid sizes). */
size_t sgdb_step_host_workspace_bytes(sgdb_dtype_t dt, int64_t P, int64_t ld, int32_t N, int32_t b);

/*
 * sgdb_step_host_static -- sgdb_step_host for callers that have no device memory
 * to hand over and must not create any.  (The paper has no counterpart; this is a
 * deployment convenience.)
 *
 * Who needs it: a server loop that runs after the process has given every byte of
 * device memory to another component's pool; code that runs where cudaMalloc is
 * off limits because it may fail under a memory budget or stalls the whole device
 * while it runs; a plug-in that is handed tensors but no allocator.  Such callers
 * still own the inputs and outputs, but cannot supply sgdb_step_host's workspace.
 *
 * Here the workspace is a fixed array of SGDB_STATIC_SCRATCH_BYTES that is part of
 * the library image: every GPU that loads the library holds it until the process
 * exits.  The call allocates and frees nothing, neither directly nor through a
 * library routine.  Arguments and results are exactly those of sgdb_step_host
 * without the two workspace arguments.
 *
 *   - Sizes whose workspace (sgdb_step_host_workspace_bytes) exceeds
 *     SGDB_STATIC_SCRATCH_BYTES are refused with SGDB_ERR_UNSUPPORTED and a line
 *     on stderr; nothing is launched.
 *   - The first call on each device looks up the array's device address (with that
 *     device current) and keeps it; make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the last
 *     call left in it.  Nothing in it needs to start at zero: every byte the
 *     kernels read is written by this call's own copies first.  Two calls that
 *     overlap on the same device (different streams or threads) race on it: keep
 *     them ordered.
 */
#define SGDB_STATIC_SCRATCH_BYTES (8u << 20)
sgdb_status_t sgdb_step_host_static(const void *h_grad, sgdb_dtype_t dt, int64_t P, int64_t ld,
                                    const float *h_arrival, const int32_t *h_tags, int32_t t,
                                    int32_t N, int32_t b, float *d_theta, float *d_state0,
                                    float *d_state1, const sgdb_opt_t *opt, float *h_theta_out,
                                    uint8_t *h_mask, int32_t *h_order, int32_t *h_info,
                                    void *stream);

/*
 * sgdb_set_tuning -- launch-shape knobs of the row-streaming kernels, for
 * measurement sweeps (no counterpart in the paper).  stages: depth of the
 * shared-memory ring of row slices; ctas_per_sm: resident blocks per SM.
 * A value <= 0 restores that knob's default.  Affects later calls of this process.
 */
sgdb_status_t sgdb_set_tuning(int32_t stages, int32_t ctas_per_sm);

/*
 * sgdb_set_wait_limit_ns -- patience of the waits inside the row-streaming kernels (no counterpart in the
 * paper).  Every wait of those kernels on a shared-memory barrier gives up after this many nanoseconds of wall
 * time; the kernel then stops, waits for the copies it still has in flight, reports SGDB_ERR_TIMEOUT in
 * d_info[1] and ends normally -- theta and state may then be updated in part and must be considered lost.
 * Default 2 s, which no correct run comes near (a wait lasts microseconds).  A negative value restores the
 * default; 0 means no patience at all -- a wait whose data is not there yet gives up at once, which happens
 * in every launch (used by the tests to show on the device that the path works); values above 10 s are refused.  Affects later calls of this process.
 */
sgdb_status_t sgdb_set_wait_limit_ns(int64_t limit_ns);

/*
 * sgdb_set_arrival_tuning -- launch-shape knobs of sgdb_accumulate_arrival (no counterpart
 * in the paper).  resident_bytes: how many leading bytes of the running sum d_acc the
 * kernels ask the L2 cache to keep between one arrival's launch and the next (the sum is
 * written by one launch and read by the following one; the gradient rows always stream
 * through).  0 streams the whole sum; a negative value restores the default.
 * blocks_per_sm: resident blocks per SM, <= 0 restores the default.  Results do not depend
 * on either knob.  Affects later calls of this process.
 */
sgdb_status_t sgdb_set_arrival_tuning(int64_t resident_bytes, int32_t blocks_per_sm);

/*
 * sgdb_selftest_bounded_wait -- shows on the device that a wait inside the kernels cannot hang (no
 * counterpart in the paper).  Every on-chip wait of the row-streaming kernels is bounded by wall time and
 * ends in SGDB_ERR_TIMEOUT; in a correct run that never happens, so this call exercises the same wait
 * routine on a barrier that nothing will ever complete: one small block waits for `limit_ns`
 * (0 .. 100 ms, larger values are refused), gives up, and the kernel ends normally.
 *   d_out [3] int32 out: {SGDB_ERR_TIMEOUT, nanoseconds waited, 1 if a second waiter was released by the
 *                         first one's give-up}
 */
sgdb_status_t sgdb_selftest_bounded_wait(int64_t limit_ns, int32_t *d_out, void *stream);

const char *sgdb_strerror(sgdb_status_t status); /* static string, never NULL */
int sgdb_version(void);                          /* major*10000 + minor*100 + patch */

#ifdef __cplusplus
}
#endif
#endif /* SGDB_H_ */
