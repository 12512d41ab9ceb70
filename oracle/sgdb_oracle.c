/*
 * sgdb_oracle.c -- plain CPU statement of the synchronous parameter-server step
 * with backup workers, in fp64.
 *
 * THIS IS TEST INFRASTRUCTURE.  It exists so that the CUDA library can be checked
 * against something written straight from the paper.  It is slow on purpose:
 * single-threaded, one loop per sentence of the method, no blocking, no fusion.
 * It shares no code, header or table with the CUDA library and neither includes
 * the other.  Only tests, the smoke check and the CPU-baseline leg of the
 * benchmark may call it.
 *
 * Source: "Revisiting Distributed Synchronous SGD" (arXiv 1604.00981).
 *   Section 3      -- N + b workers are started; the first N gradients to arrive
 *                     are used, the slowest b are dropped when they arrive.
 *   Algorithm 4    -- the server's loop: G = {}; while |G| < N: receive (G, t');
 *                     keep it iff t' == t; then theta <- theta - gamma_t/N * sum G.
 *   Section 1.1    -- SGD rule; "update equations differ" for the other rules.
 *   Appendix A     -- RMSProp with momentum (decay 0.9, momentum 0.9).
 *
 * Readings taken where the paper is silent (each also listed in the design notes):
 *   - two gradients with equal arrival time: the lower worker id arrives first;
 *   - arrival NaN or +-inf: that gradient never arrives;
 *   - tag t' > t is dropped like t' < t (Algorithm 4 tests equality);
 *   - fewer than N current gradients: the server cannot finish the iteration;
 *     the oracle reports ORACLE_INSUFFICIENT and changes nothing;
 *   - arrival times are compared as fp32 values, the type they are given in;
 *   - optimizer equations (the paper prints only SGD's): see oracle_update.
 *     PARITY UNPINNED BY THE PAPER for momentum / RMSProp / Adam: no equation or
 *     worked number is printed there; the forms below are pinned by closed forms
 *     that hold for the chosen reading only.
 *   - two-level aggregation (Section 6 names it, nothing more): see oracle_select_grouped.
 *     PARITY UNPINNED BY THE PAPER; pinned by a replay of machines and messages, by its
 *     reduction to Algorithm 4 with one worker per machine, and by library means.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_OK = 0, ORACLE_INVALID = 1, ORACLE_INSUFFICIENT = 2 };
enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };
enum { ORACLE_SGD = 0, ORACLE_MOMENTUM = 1, ORACLE_RMSPROP = 2, ORACLE_ADAM = 3, ORACLE_ADAGRAD = 4 };

typedef struct {
  int32_t kind;
  double lr, momentum, decay, beta1, beta2, eps;
  int64_t step; /* 1-based count of updates, this one included (Adam) */
} oracle_opt_t;

/* A bf16 value is the upper 16 bits of an fp32 value; widening is exact. */
static double bf16_bits_to_double(uint16_t bits) {
  uint32_t u = ((uint32_t)bits) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

static double grad_at(const void *grad, int dtype, int64_t index) {
  if (dtype == ORACLE_BF16) return bf16_bits_to_double(((const uint16_t *)grad)[index]);
  return (double)((const float *)grad)[index];
}

/* worker a reaches the server before worker b */
static int arrives_before(const float *arrival, int32_t a, int32_t b) {
  if (arrival[a] < arrival[b]) return 1;
  if (arrival[a] > arrival[b]) return 0;
  return a < b;
}

/*
 * Section 3 + Algorithm 4 (the while loop): the gradients the server ends up
 * with are the first N to arrive among those tagged t.  Written as its plain
 * definition: list the valid workers, put them in arrival sequence (insertion
 * sort), take the first N.
 *   mask [W]  1 for a kept worker;  order [N] kept ids in arrival sequence;
 *   n_valid   number of workers with tag == t and a finite arrival time.
 */
int oracle_select(const float *arrival, const int32_t *tags, int32_t t, int32_t N, int32_t b,
                  uint8_t *mask, int32_t *order, int32_t *n_valid) {
  if (N < 1 || b < 0) return ORACLE_INVALID;
  int32_t W = N + b;
  int32_t *seq = (int32_t *)malloc(sizeof(int32_t) * (size_t)W);
  int32_t count = 0;
  for (int32_t w = 0; w < W; ++w) {
    if (tags[w] != t) continue;         /* Algorithm 4: t' == t or the gradient is dropped */
    if (!isfinite(arrival[w])) continue; /* never arrives */
    int32_t pos = count++;
    while (pos > 0 && arrives_before(arrival, w, seq[pos - 1])) {
      seq[pos] = seq[pos - 1];
      --pos;
    }
    seq[pos] = w;
  }
  *n_valid = count;
  if (count < N) {
    free(seq);
    return ORACLE_INSUFFICIENT;
  }
  for (int32_t w = 0; w < W; ++w) mask[w] = 0;
  for (int32_t k = 0; k < N; ++k) { /* the server stops waiting at |G| = N */
    order[k] = seq[k];
    mask[seq[k]] = 1;
  }
  free(seq);
  return ORACLE_OK;
}

/*
 * The alternative the paper names in its conclusion: a time-out instead of backup
 * workers.  The paper gives no algorithm for it; the reading taken here is the direct
 * counterpart of Algorithm 4: the server waits until `deadline`, keeps every gradient
 * tagged t that has arrived by then (arrival <= deadline), drops the rest, and averages
 * over the n it kept.  n_min >= 1 is the fewest it accepts; with fewer the iteration
 * cannot complete and nothing changes.  PARITY UNPINNED BY THE PAPER (no definition
 * printed); pinned by brute force and by its reductions to Algorithm 4.
 *   mask [W], order [W] (first *n_kept entries used, arrival sequence), *n_kept.
 */
int oracle_select_deadline(const float *arrival, const int32_t *tags, int32_t t, int32_t W,
                           float deadline, int32_t n_min, uint8_t *mask, int32_t *order,
                           int32_t *n_kept) {
  if (W < 1 || n_min < 1) return ORACLE_INVALID;
  int32_t *seq = (int32_t *)malloc(sizeof(int32_t) * (size_t)W);
  int32_t count = 0;
  for (int32_t w = 0; w < W; ++w) {
    if (tags[w] != t) continue;
    if (!isfinite(arrival[w])) continue;
    if (!(arrival[w] <= deadline)) continue; /* still on its way when the server stops waiting */
    int32_t pos = count++;
    while (pos > 0 && arrives_before(arrival, w, seq[pos - 1])) {
      seq[pos] = seq[pos - 1];
      --pos;
    }
    seq[pos] = w;
  }
  *n_kept = count;
  if (count < n_min) {
    free(seq);
    return ORACLE_INSUFFICIENT;
  }
  for (int32_t w = 0; w < W; ++w) mask[w] = 0;
  for (int32_t k = 0; k < count; ++k) {
    order[k] = seq[k];
    mask[seq[k]] = 1;
  }
  free(seq);
  return ORACLE_OK;
}

/* One iteration with the time-out rule: mean over the n kept gradients, then the update. */
int oracle_step_deadline(const void *grad, int dtype, int64_t P, int64_t ld, const float *arrival,
                         const int32_t *tags, int32_t t, int32_t W, float deadline, int32_t n_min,
                         double *theta, double *s0, double *s1, const oracle_opt_t *opt,
                         uint8_t *mask, int32_t *order, int32_t *n_kept);

/* Algorithm 4's update line, the part before the learning rate: (1/N) sum_{G in set} G. */
int oracle_aggregate(const void *grad, int dtype, int64_t P, int64_t ld, int32_t N,
                     const int32_t *order, double *mean) {
  if (N < 1 || P < 0 || ld < P) return ORACLE_INVALID;
  for (int64_t i = 0; i < P; ++i) {
    double sum = 0.0;
    for (int32_t k = 0; k < N; ++k) sum += grad_at(grad, dtype, (int64_t)order[k] * ld + i);
    mean[i] = sum / (double)N;
  }
  return ORACLE_OK;
}

/*
 * The update of theta from the mean gradient g.
 *   SGD       theta <- theta - lr*g                          (Section 1.1; Algorithm 4 with
 *                                                             lr = gamma_t, g = sum/N)
 *   momentum  v <- mu*v + g;  theta <- theta - lr*v
 *   RMSProp   s <- rho*s + (1-rho)*g^2;  m <- mu*m + lr*g/sqrt(s+eps);  theta <- theta - m
 *             (Appendix A: "RMSProp with momentum", decay rho, momentum mu)
 *   Adam      m <- b1*m + (1-b1)*g;  v <- b2*v + (1-b2)*g^2;
 *             theta <- theta - lr * (m/(1-b1^k)) / (sqrt(v/(1-b2^k)) + eps),  k = step
 *   AdaGrad   s <- s + g^2;  theta <- theta - lr * g / (sqrt(s) + eps)
 *             (named in the Introduction next to RMSProp and Adam; Duchi et al.'s rule)
 * s0/s1 hold (v,-), (s,m), (m,v), (s,-) for momentum, RMSProp, Adam, AdaGrad.
 */
int oracle_update(double *theta, double *s0, double *s1, const double *mean, int64_t P,
                  const oracle_opt_t *opt) {
  for (int64_t i = 0; i < P; ++i) {
    double g = mean[i];
    switch (opt->kind) {
      case ORACLE_SGD:
        theta[i] = theta[i] - opt->lr * g;
        break;
      case ORACLE_MOMENTUM:
        s0[i] = opt->momentum * s0[i] + g;
        theta[i] = theta[i] - opt->lr * s0[i];
        break;
      case ORACLE_RMSPROP:
        s0[i] = opt->decay * s0[i] + (1.0 - opt->decay) * g * g;
        s1[i] = opt->momentum * s1[i] + opt->lr * g / sqrt(s0[i] + opt->eps);
        theta[i] = theta[i] - s1[i];
        break;
      case ORACLE_ADAM: {
        s0[i] = opt->beta1 * s0[i] + (1.0 - opt->beta1) * g;
        s1[i] = opt->beta2 * s1[i] + (1.0 - opt->beta2) * g * g;
        double m_hat = s0[i] / (1.0 - pow(opt->beta1, (double)opt->step));
        double v_hat = s1[i] / (1.0 - pow(opt->beta2, (double)opt->step));
        theta[i] = theta[i] - opt->lr * m_hat / (sqrt(v_hat) + opt->eps);
        break;
      }
      case ORACLE_ADAGRAD:
        s0[i] = s0[i] + g * g;
        theta[i] = theta[i] - opt->lr * g / (sqrt(s0[i]) + opt->eps);
        break;
      default:
        return ORACLE_INVALID;
    }
  }
  return ORACLE_OK;
}

/* One iteration of Algorithm 4's outer loop: select, aggregate, update. */
int oracle_step(const void *grad, int dtype, int64_t P, int64_t ld, const float *arrival,
                const int32_t *tags, int32_t t, int32_t N, int32_t b, double *theta, double *s0,
                double *s1, const oracle_opt_t *opt, uint8_t *mask, int32_t *order,
                int32_t *n_valid) {
  int rc = oracle_select(arrival, tags, t, N, b, mask, order, n_valid);
  if (rc != ORACLE_OK) return rc;
  double *mean = (double *)malloc(sizeof(double) * (size_t)(P > 0 ? P : 1));
  rc = oracle_aggregate(grad, dtype, P, ld, N, order, mean);
  if (rc == ORACLE_OK) rc = oracle_update(theta, s0, s1, mean, P, opt);
  free(mean);
  return rc;
}

int oracle_step_deadline(const void *grad, int dtype, int64_t P, int64_t ld, const float *arrival,
                         const int32_t *tags, int32_t t, int32_t W, float deadline, int32_t n_min,
                         double *theta, double *s0, double *s1, const oracle_opt_t *opt,
                         uint8_t *mask, int32_t *order, int32_t *n_kept) {
  int rc = oracle_select_deadline(arrival, tags, t, W, deadline, n_min, mask, order, n_kept);
  if (rc != ORACLE_OK) return rc;
  double *mean = (double *)malloc(sizeof(double) * (size_t)(P > 0 ? P : 1));
  rc = oracle_aggregate(grad, dtype, P, ld, *n_kept, order, mean); /* divisor: the number kept */
  if (rc == ORACLE_OK) rc = oracle_update(theta, s0, s1, mean, P, opt);
  free(mean);
  return rc;
}

/*
 * Section 1.1 / the last line of Algorithm 4: the exponential moving average of the
 * parameters, avg(t) = alpha * avg(t-1) + (1 - alpha) * theta(t).  The paper does not
 * define avg(-1); the caller initialises it (the tests use theta(0)).
 */
void oracle_ema(double *avg, const double *theta, int64_t P, double alpha) {
  for (int64_t i = 0; i < P; ++i) avg[i] = alpha * avg[i] + (1.0 - alpha) * theta[i];
}

/*
 * One iteration of Algorithm 4 including its last line.  As printed, iteration t
 * computes theta(t+1) from theta(t) and then averages theta(t): the average sees
 * the parameters as they were before this iteration's update.
 */
int oracle_step_ema(const void *grad, int dtype, int64_t P, int64_t ld, const float *arrival,
                    const int32_t *tags, int32_t t, int32_t N, int32_t b, double *theta, double *s0,
                    double *s1, const oracle_opt_t *opt, double *avg, double alpha, uint8_t *mask,
                    int32_t *order, int32_t *n_valid) {
  double *theta_t = (double *)malloc(sizeof(double) * (size_t)(P > 0 ? P : 1));
  memcpy(theta_t, theta, sizeof(double) * (size_t)P);
  int rc = oracle_step(grad, dtype, P, ld, arrival, tags, t, N, b, theta, s0, s1, opt, mask, order, n_valid);
  if (rc == ORACLE_OK) oracle_ema(avg, theta_t, P, alpha);
  free(theta_t);
  return rc;
}

/*
 * Appendix A.2 / A.3: learning rate after t iterations, gamma0 * beta^(t N / (2 T)) with
 * T = |X| / B mini-batches in the data set; N = 1 is the asynchronous schedule.
 */
double oracle_learning_rate(double gamma0, double beta, int64_t t, int64_t N, double T) {
  return gamma0 * pow(beta, (double)t * (double)N / (2.0 * T));
}

/*
 * Algorithm 4's while loop, one received gradient per call.
 *   state[0] = |G| so far, state[1] = gradients received so far,
 *   state[2] = lowest iteration still open (the server's own t).
 * Returns through *outcome: 0 dropped, 1 added to the set, 2 added and theta updated.
 * A gradient is kept iff its tag equals t, iteration t is still open and |G| < N.
 * On the N-th kept gradient the server updates theta, empties the set and moves
 * on to t + 1, so anything that still arrives for t is dropped (Section 3).
 */
int oracle_accumulate_arrival(const void *row, int dtype, int32_t row_tag, int32_t t, int32_t N,
                              int64_t P, double *acc, int32_t *state, double *theta, double *s0,
                              double *s1, const oracle_opt_t *opt, int32_t *outcome);

/* The same with Algorithm 4's last line: when the N-th gradient triggers the update, the average takes in
 * the parameters as they were before it (avg may be NULL: no average is kept). */
int oracle_accumulate_arrival_ema(const void *row, int dtype, int32_t row_tag, int32_t t, int32_t N,
                                  int64_t P, double *acc, int32_t *state, double *theta, double *s0,
                                  double *s1, const oracle_opt_t *opt, double *avg, double alpha,
                                  int32_t *outcome) {
  double *theta_t = (double *)malloc(sizeof(double) * (size_t)(P > 0 ? P : 1));
  memcpy(theta_t, theta, sizeof(double) * (size_t)P);
  int rc = oracle_accumulate_arrival(row, dtype, row_tag, t, N, P, acc, state, theta, s0, s1, opt, outcome);
  if (rc == ORACLE_OK && *outcome == 2 && avg != NULL) oracle_ema(avg, theta_t, P, alpha);
  free(theta_t);
  return rc;
}

int oracle_accumulate_arrival(const void *row, int dtype, int32_t row_tag, int32_t t, int32_t N,
                              int64_t P, double *acc, int32_t *state, double *theta, double *s0,
                              double *s1, const oracle_opt_t *opt, int32_t *outcome) {
  if (N < 1 || P < 0) return ORACLE_INVALID;
  state[1] += 1;
  if (row_tag != t || t < state[2] || state[0] >= N) {
    *outcome = 0;
    return ORACLE_OK;
  }
  if (state[0] == 0)
    for (int64_t i = 0; i < P; ++i) acc[i] = 0.0; /* G = {} */
  for (int64_t i = 0; i < P; ++i) acc[i] += grad_at(row, dtype, i);
  state[0] += 1;
  *outcome = 1;
  if (state[0] == N) {
    for (int64_t i = 0; i < P; ++i) acc[i] = acc[i] / (double)N;
    int rc = oracle_update(theta, s0, s1, acc, P, opt);
    if (rc != ORACLE_OK) return rc;
    state[0] = 0;
    state[2] = t + 1;
    *outcome = 2;
  }
  return ORACLE_OK;
}

/*
 * Two-level aggregation.  The paper's conclusion (Section 6) names it in one sentence: the
 * gradients of workers that share a machine are combined before they are sent to the
 * parameter server.  It prints no algorithm.  PARITY UNPINNED BY THE PAPER; the reading
 * taken here keeps Algorithm 4 as it is and lets a machine play the part of a worker:
 *   - worker w runs on machine group[w], 0 <= group[w] < M;
 *   - a machine's message is the mean of its workers' gradients (the gradient of its
 *     combined mini-batch); it can only be sent when the slowest of them is done, so it
 *     arrives at the maximum of their arrival times;
 *   - the message counts for iteration t only if every one of its workers computed its
 *     gradient for t and every arrival time is finite; a machine without workers sends
 *     nothing;
 *   - the server runs Algorithm 4 over messages: the first N to arrive are used (equal
 *     times: lower machine id first), the rest dropped, and theta moves by the mean of the
 *     N messages.
 * Outputs: mask [W] 1 for every worker whose gradient is used; group_order [N] the kept
 * machines in arrival sequence; order [W], of which the first *n_rows entries are the used
 * workers machine by machine in that sequence and, within a machine, in the order their
 * gradients were ready (arrival, then id); *n_valid the number of machines whose message
 * counts.
 */
int oracle_select_grouped(const float *arrival, const int32_t *tags, const int32_t *group, int32_t t,
                          int32_t W, int32_t M, int32_t N, uint8_t *mask, int32_t *group_order,
                          int32_t *order, int32_t *n_rows, int32_t *n_valid) {
  if (W < 1 || M < 1 || N < 1) return ORACLE_INVALID;
  for (int32_t w = 0; w < W; ++w)
    if (group[w] < 0 || group[w] >= M) return ORACLE_INVALID;
  float *sent_at = (float *)malloc(sizeof(float) * (size_t)M);
  int32_t *seq = (int32_t *)malloc(sizeof(int32_t) * (size_t)M);
  int32_t count = 0;
  for (int32_t g = 0; g < M; ++g) {
    int32_t members = 0, counts = 1;
    float latest = 0.0f;
    for (int32_t w = 0; w < W; ++w) {
      if (group[w] != g) continue;
      if (tags[w] != t || !isfinite(arrival[w])) counts = 0;
      if (members == 0 || arrival[w] > latest) latest = arrival[w];
      ++members;
    }
    if (members == 0 || !counts) continue;
    sent_at[g] = latest; /* the machine waits for its slowest worker */
    int32_t pos = count++;
    while (pos > 0 && arrives_before(sent_at, g, seq[pos - 1])) {
      seq[pos] = seq[pos - 1];
      --pos;
    }
    seq[pos] = g;
  }
  *n_valid = count;
  if (count < N) {
    free(sent_at);
    free(seq);
    return ORACLE_INSUFFICIENT;
  }
  for (int32_t w = 0; w < W; ++w) mask[w] = 0;
  int32_t rows = 0;
  for (int32_t k = 0; k < N; ++k) {
    int32_t g = seq[k];
    group_order[k] = g;
    int32_t first = rows;
    for (int32_t w = 0; w < W; ++w) {
      if (group[w] != g) continue;
      mask[w] = 1;
      int32_t pos = rows++;
      while (pos > first && arrives_before(arrival, w, order[pos - 1])) {
        order[pos] = order[pos - 1];
        --pos;
      }
      order[pos] = w;
    }
  }
  *n_rows = rows;
  free(sent_at);
  free(seq);
  return ORACLE_OK;
}

/* One server iteration over machine messages: select, form each kept machine's message (the
 * mean of its workers' gradients), average the N messages, update. */
int oracle_step_grouped(const void *grad, int dtype, int64_t P, int64_t ld, const float *arrival,
                        const int32_t *tags, const int32_t *group, int32_t t, int32_t W, int32_t M,
                        int32_t N, double *theta, double *s0, double *s1, const oracle_opt_t *opt,
                        uint8_t *mask, int32_t *group_order, int32_t *order, int32_t *n_rows,
                        int32_t *n_valid) {
  if (P < 0 || ld < P) return ORACLE_INVALID;
  int rc = oracle_select_grouped(arrival, tags, group, t, W, M, N, mask, group_order, order, n_rows, n_valid);
  if (rc != ORACLE_OK) return rc;
  double *mean = (double *)malloc(sizeof(double) * (size_t)(P > 0 ? P : 1));
  for (int64_t i = 0; i < P; ++i) {
    double total = 0.0;
    for (int32_t k = 0; k < N; ++k) {
      double message = 0.0;
      int32_t members = 0;
      for (int32_t w = 0; w < W; ++w) {
        if (group[w] != group_order[k]) continue;
        message += grad_at(grad, dtype, (int64_t)w * ld + i);
        ++members;
      }
      total += message / (double)members;
    }
    mean[i] = total / (double)N;
  }
  rc = oracle_update(theta, s0, s1, mean, P, opt);
  free(mean);
  return rc;
}

/*
 * The time-out rule (see oracle_select_deadline) one received gradient at a time.  The server
 * listens until `deadline`: a gradient joins the set iff it is tagged t, iteration t is still
 * open and it arrived (finite time) by the deadline; there is no upper count.  When the
 * deadline has passed the server closes the iteration (oracle_accumulate_close): with at least
 * n_min gradients in the set it moves theta by their mean (divisor: the number in the set),
 * empties the set and opens t + 1; with fewer the iteration does not complete and nothing
 * changes.  state as in oracle_accumulate_arrival.  PARITY UNPINNED BY THE PAPER, like the
 * batched time-out rule it must agree with.
 * *outcome: 0 dropped, 1 added.
 */
int oracle_accumulate_arrival_deadline(const void *row, int dtype, int32_t row_tag, float row_arrival,
                                       int32_t t, float deadline, int64_t P, double *acc,
                                       int32_t *state, int32_t *outcome) {
  if (P < 0) return ORACLE_INVALID;
  state[1] += 1;
  if (row_tag != t || t < state[2] || !isfinite(row_arrival) || !(row_arrival <= deadline)) {
    *outcome = 0;
    return ORACLE_OK;
  }
  if (state[0] == 0)
    for (int64_t i = 0; i < P; ++i) acc[i] = 0.0; /* G = {} */
  for (int64_t i = 0; i < P; ++i) acc[i] += grad_at(row, dtype, i);
  state[0] += 1;
  *outcome = 1;
  return ORACLE_OK;
}

/* The deadline of iteration t has passed.  *outcome: 2 theta updated, 0 nothing done (t was closed
 * already).  Returns ORACLE_INSUFFICIENT, with nothing changed, when fewer than n_min gradients are
 * in the set.  avg may be NULL; otherwise it takes in theta as it was before the update. */
int oracle_accumulate_close(int32_t t, int32_t n_min, int64_t P, double *acc, int32_t *state,
                            double *theta, double *s0, double *s1, const oracle_opt_t *opt,
                            double *avg, double alpha, int32_t *outcome) {
  if (n_min < 1 || P < 0) return ORACLE_INVALID;
  *outcome = 0;
  if (t < state[2]) return ORACLE_OK;
  if (state[0] < n_min) return ORACLE_INSUFFICIENT;
  if (avg != NULL) oracle_ema(avg, theta, P, alpha); /* theta is still theta(t) here */
  for (int64_t i = 0; i < P; ++i) acc[i] = acc[i] / (double)state[0];
  int rc = oracle_update(theta, s0, s1, acc, P, opt);
  if (rc != ORACLE_OK) return rc;
  state[0] = 0;
  state[2] = t + 1;
  *outcome = 2;
  return ORACLE_OK;
}
