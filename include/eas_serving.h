/*
 * eas_serving.h -- host-side control logic around the Encode stage (plain C ABI, no device code).
 *
 * The paper wraps the encoder forward pass in three O(1) runtime mechanisms: a load-adaptive micro-batcher
 * (Section 3.2), a rate-controlled offload router with per-destination envelopes (Section 3.3) and a lookup table that
 * picks the SM share per micro-batch (Section 3.4).  They decide WHEN a micro-batch is dispatched, WHERE its embeddings
 * go and on HOW MANY SMs eas_encode_microbatch runs.  All functions are pure host code; every pointer is a host pointer.
 */
#ifndef EAS_SERVING_H_
#define EAS_SERVING_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- Section 3.2, Eq. 5: Poisson-gap dispatch rule ---------------------------------------------------------------- */

/* kappa = -ln(1 - p^(1/(B-1))): with Poisson arrivals of rate lambda, a batch whose B-1 successive gaps are all at most
 * g = kappa / lambda fills to B with probability p.  B <= 1 returns 0 (dispatch immediately); p outside (0,1) returns NaN. */
double eas_poisson_gap_kappa(int32_t batch_bound, double fill_probability);

typedef struct eas_batcher eas_batcher; /* opaque; created and destroyed by the library (host memory only) */

/* batch_bound B >= 1; arrival_rate lambda > 0 (requests per second reaching this encode worker); fill_probability p in
 * (0,1) (the paper uses 0.6); max_age A > 0 seconds (the paper uses 1.0).  Returns NULL on a bad argument. */
eas_batcher* eas_batcher_create(int32_t batch_bound, double arrival_rate, double fill_probability, double max_age);
void eas_batcher_destroy(eas_batcher* b);
double eas_batcher_gap(const eas_batcher* b); /* g = kappa / lambda, seconds */

/* Time at which the open micro-batch dispatches if nothing else arrives: min(last arrival + g, first arrival + A);
 * +infinity when no request is waiting. */
double eas_batcher_deadline(const eas_batcher* b);

/* A request arrives at time t (seconds, non-decreasing across calls).  Up to two micro-batches can leave: the open one
 * if its deadline passed before t (dispatch time = that deadline), and the one this request completes (size B, time t).
 * sizes/times: host arrays of 2.  Returns the number of dispatches written (0, 1 or 2), -1 on a bad argument. */
int32_t eas_batcher_on_arrival(eas_batcher* b, double t, int32_t* sizes, double* times);

/* Timer check at time `now`: dispatches the open micro-batch if idle > g or age > A.  Returns 1 and writes size/time, or 0. */
int32_t eas_batcher_on_timer(eas_batcher* b, double now, int32_t* size, double* time);

/* ---- Section 3.3: deficit-counter router and per-destination envelopes -------------------------------------------- */

/* Accumulator d starts at 0; each request adds s; if d >= 1 the request goes to the remote path and d drops by 1.
 * The ratio is held as an exact fraction num/den so that, e.g., s = 7/10 reproduces the paper's Figure 6 (a binary
 * floating-point accumulator does not: ten times 0.7 falls just short of 7). */
typedef struct {
  int64_t num, den; /* s = num / den, 0 <= num <= den, den > 0 */
  int64_t acc;      /* d * den, always in [0, den) between requests */
} eas_router;

int32_t eas_router_init(eas_router* r, int64_t s_num, int64_t s_den);                  /* 0 ok, -1 bad ratio */
int32_t eas_router_init_from_double(eas_router* r, double s, int64_t max_denominator); /* closest fraction with den <= max */
int32_t eas_router_next(eas_router* r);                                                /* 1 = remote, 0 = local */

/* Envelope plan: requests of one micro-batch are grouped per destination into one contiguous tensor each, so that a
 * micro-batch issues at most one transfer per destination.  dest[i] in [0, n_dest) and rows[i] (embedding rows of request
 * i) are inputs; row_offset[i] receives the first row of request i inside its destination's envelope (requests keep their
 * arrival order inside an envelope); dest_rows[k] receives the envelope's total rows.  Returns 0, or -1 on a bad argument. */
int32_t eas_envelope_plan(const int32_t* dest, const int32_t* rows, int32_t n_requests, int32_t n_dest,
                          int64_t* row_offset, int64_t* dest_rows);

/* Encode order that lays the envelopes out back to back in the encoder's output.  The encoder writes the embedding rows
 * of its items in the order the items are listed, and items do not interact (block-diagonal attention), so listing the
 * requests of a micro-batch grouped by destination makes the final epilogue itself write every request into its
 * destination's contiguous envelope: no gather after the forward pass.  order[k] receives the index of the request to list
 * k-th (a stable sort by destination, so arrival order is kept inside an envelope, as in eas_envelope_plan);
 * env_first_row[d] receives the first output row of destination d's envelope.  Request i then occupies rows
 * [env_first_row[dest[i]] + row_offset[i], + rows[i]) of out_embeddings.  Returns 0, or -1 on a bad argument. */
int32_t eas_envelope_order(const int32_t* dest, const int32_t* rows, int32_t n_requests, int32_t n_dest, int32_t* order,
                           int64_t* env_first_row);

/* ---- Section 3.4: SM lookup table ---------------------------------------------------------------------------------- */

enum { EAS_SM_TABLE_MAX_LEVELS = 16 };
typedef struct {
  int32_t n_levels;
  int32_t sm_count[EAS_SM_TABLE_MAX_LEVELS];  /* SMs of each level, ascending */
  int32_t max_batch[EAS_SM_TABLE_MAX_LEVELS]; /* largest micro-batch the level sustains (0: none) */
} eas_sm_table;

/* Built once from an encode-only latency sweep: latency[l * n_batches + b] is the forward-pass latency of batch size
 * batches[b] on sm_counts[l] SMs, exclusive[b] the latency with the whole GPU.  A level sustains a batch size when its
 * latency is at most (1 + tolerance) times the exclusive one (the paper uses 20 %); max_batch is the largest such size
 * for which all smaller profiled sizes are sustained too.  sm_counts ascending, batches ascending.  Returns 0 or -1. */
int32_t eas_sm_table_build(const int32_t* sm_counts, int32_t n_levels, const int32_t* batches, int32_t n_batches,
                           const double* latency, const double* exclusive, double tolerance, eas_sm_table* out);

/* Smallest level whose sustained batch size covers `batch`; the largest level if none does.  Returns its SM count
 * (the value to pass as sm_budget), or -1 on a bad table. */
int32_t eas_sm_table_lookup(const eas_sm_table* t, int32_t batch);

/* ---- Section 3.1, Algorithm 1 lines 1-12, Eq. 3 and Eq. 4: Stage 1 of the configuration search ------------------- */

/* One candidate allocation of workers to stages and what Stage 1 derives for it. */
typedef struct {
  int32_t n_encode, n_prefill, n_decode; /* workers per stage (inputs) */
  int32_t n_local;                       /* co-resident local prefill workers on encode GPUs (input) */
  double rho_e, rho_p, rho_d;            /* utilisations: (Lambda/n)/C; prefill: Lambda / (C_P (n_P + n_L alpha)) */
  double score;                          /* max of the three */
  int32_t b_max;                         /* ceil(Lambda / n_E): cap of the batch bound B for Stage 2 */
  double s_star;                         /* n_P / (n_P + n_L alpha): centre of the offload-ratio window (+-0.2) */
  int32_t kept;                          /* 1 if the allocation survives all three filters */
} eas_has_candidate;

/* Scores every candidate in place, discards score >= 1, prunes score > prune_factor x the minimum surviving score
 * (1.2 in the paper), keeps the top_k best (3 in the paper; ties keep the earlier candidate).  c_e, c_p, c_d: profiled
 * per-worker capacities in requests/s; alpha in [0,1]: memory share of a local prefill worker.  Returns the number
 * kept, or -1 on a bad argument. */
int32_t eas_has_stage1(eas_has_candidate* cand, int32_t n_candidates, double target_rate, double c_e, double c_p,
                       double c_d, double alpha, double prune_factor, int32_t top_k);

#ifdef __cplusplus
}
#endif
#endif /* EAS_SERVING_H_ */
