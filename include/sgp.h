/*
 * sgp.h -- C ABI of the fused Stochastic Gradient Push (SGP) step for n simulated nodes
 *          stacked on one NVIDIA B200 (sm_100a).
 *
 * State (all fp32, owned by the caller, DEVICE memory unless a name starts with h_):
 *   X  n x ld   push-sum numerators x_i            (row i = node i, ld >= d floats between rows)
 *   W  n        push-sum weights w_i               (w_i^(0) = 1)
 *   M  n x ld   momentum buffers u_i               (never mixed; u^(0) = 0)
 *   G  n x ld   stochastic gradients of step k, evaluated by the caller at Z
 *   Z  n x ld   de-biased parameters z_i = x_i / w_i
 * Convention for the mixing matrix P^(k): p_ij is the weight RECEIVER i applies to SENDER j
 * (rows = receivers, columns = senders), every node is its own in/out-neighbour, columns sum to 1
 * (Sec. 2 "Approximate distributed averaging"; supplementary "Modeling message delays").
 *
 * Layout advice: make ld a multiple of 256 floats so that every row starts on a 1 KB boundary; the step then
 * runs at ~0.98 of the device's copy bandwidth instead of ~0.91 with a dense pitch ld = d whose rows start off
 * the 128-byte grid.
 *
 * Every function returns an int status (SGP_OK = 0, negative = error), never throws, aborts or prints.
 * Kernels are enqueued on the caller's stream (a cudaStream_t passed as void*) and the calls return
 * without synchronising unless stated.  No call falls back to the CPU.
 */
#ifndef SGP_H_
#define SGP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SGP_OK            0
#define SGP_ERR_ARG      -1   /* bad size, null pointer, misaligned pointer, k < 0, ...               */
#define SGP_ERR_GRAPH    -2   /* schedule is not a valid column-stochastic digraph with self-loops    */
#define SGP_ERR_CUDA     -3   /* a CUDA runtime call failed; see sgp_last_cuda_error                  */
#define SGP_ERR_ALLOC    -4   /* host or device allocation failed                                     */
#define SGP_ERR_STATE    -5   /* call not valid for this handle (ring export with tau = 0; the current
                                 CUDA device is not the one the handle was created on)               */
#define SGP_ERR_DEVICE   -6   /* a kernel reported a bounded wait that ran out (status word non-zero) */
#define SGP_ERR_ZERO_WEIGHT -7 /* a push-sum weight is <= 0 or not a number: z = x / w is undefined      */
#define SGP_ERR_INVARIANT -8  /* sgp_check: non-finite state, sum of weights != n, or a column sum drifted */

/* Bits of the device status word (sgp_device_status).  Kernels only ever OR bits in; sgp_reset clears it. */
#define SGP_STATUS_WAIT_TILE     1u   /* pipelined kernel: consumers gave up waiting for a tile              */
#define SGP_STATUS_WAIT_STAGE    2u   /* pipelined kernel: the producer gave up waiting for a free stage     */
#define SGP_STATUS_WAIT_DRAIN    4u   /* pipelined kernel: copies were still pending at exit                 */
#define SGP_STATUS_ZERO_WEIGHT   8u   /* a weight was <= 0 or NaN (that node's z was written as 0, never inf) */
#define SGP_STATUS_NONFINITE    16u   /* invariant check: non-finite entries in X or in the delay ring       */
#define SGP_STATUS_WEIGHT_SUM   32u   /* invariant check: sum of weights incl. in transit differs from n     */
#define SGP_STATUS_COLUMN_SUM   64u   /* invariant check: a column sum drifted from its reference            */
#define SGP_STATUS_BOUNDS      128u   /* bounds-checked build only: an index was out of range, access skipped */

#define SGP_MAX_NODES 256     /* n <= 256: one CTA keeps all n rows of a column tile on chip          */

/* Which time-varying digraph the schedule compiler expands. */
typedef enum sgp_graph_kind {
  SGP_GRAPH_EXP_PEERS     = 0, /* App. A directed exponential graph, `peers` out-neighbours per step */
  SGP_GRAPH_COMPLETE      = 1, /* every entry 1/n (Sec. 3: equivalent to AllReduce parallel SGD)     */
  SGP_GRAPH_RANDOM_OUTDEG = 2, /* hashed random digraph, out-degree ~ U{1..min(max_outdeg, n-1)}     */
  SGP_GRAPH_CUSTOM        = 3, /* explicit edge list with per-edge weights                           */
  SGP_GRAPH_BIPARTITE_EXP = 4  /* App. A undirected bipartite exponential graph (the D-PSGD topology)   */
} sgp_graph_kind;

/*
 * Schedule descriptor (plain data, HOST memory, read only during the call that takes it).
 *  EXP_PEERS : at step k node i sends to (i + 2^((k+t) mod L)) mod n, t = 0..peers-1, with
 *              L = floor(log2(n-1)) + 1 hop distances (App. A); weights 1/|N_out| incl. self (App. C).
 *  RANDOM    : `num_steps` distinct steps, then the schedule repeats; draws are a keyed integer
 *              hash of (seed, step, node, draw) so that independent implementations agree bit for bit.
 *  BIPARTITE : n even (SGP_ERR_ARG otherwise).  At step k odd node i and even node (i + hop_k) mod n exchange
 *              messages, hop_k cycling through 2^1 - 1, ..., 2^floor(log2(n-1)) - 1 (n = 2: hop 1); weights 1/2
 *              and 1/2, so P is symmetric doubly stochastic and the push-sum weights stay 1 (Sec. 4, App. A).
 *  CUSTOM    : num_edges quadruples (edge_step, edge_sender, edge_receiver, edge_weight); self-loops are
 *              listed explicitly; steps 0..num_steps-1, repeating.  Rejected with SGP_ERR_GRAPH if an
 *              index is out of range, an edge is duplicated, a weight is not finite and > 0, a
 *              self-loop is missing, or a column does not sum to 1 within 4*deg*2^-24.
 */
typedef struct sgp_graph_desc {
  int32_t  kind;         /* sgp_graph_kind                                         */
  int32_t  peers;        /* EXP_PEERS: >= 1 (paper uses 1 and 2)                   */
  int32_t  max_outdeg;   /* RANDOM_OUTDEG: >= 1                                    */
  int32_t  reserved;     /* must be 0                                              */
  uint64_t seed;         /* RANDOM_OUTDEG                                          */
  int64_t  num_steps;    /* RANDOM_OUTDEG, CUSTOM: period of the schedule (>= 1)   */
  const int32_t *edge_step;      /* CUSTOM only, host arrays of num_edges entries  */
  const int32_t *edge_sender;
  const int32_t *edge_receiver;
  const float   *edge_weight;
  int64_t  num_edges;
} sgp_graph_desc;

/* ---------------------------------------------------------------------------------------------
 * Graph-schedule compiler (host only; needs no GPU).  Turns the time-varying digraph into, for
 * every step of one period, the in-neighbour lists of P^(k) in CSR form: row i lists the senders j
 * with p_ij != 0 in ascending j (self in its sorted place) and the fp32 weights p_ij.  For the
 * uniform kinds p_ij = (float)(1.0 / |N_out_j|) (App. C).  Defines the mix x_i' = sum_j p_ij x_j
 * of Alg. 1 line 6.  The returned object is owned by the caller until sgp_schedule_destroy.
 * ------------------------------------------------------------------------------------------- */
typedef struct sgp_schedule sgp_schedule;

int sgp_schedule_compile(sgp_schedule **out, int n, const sgp_graph_desc *g);
int sgp_schedule_destroy(sgp_schedule *s);
/* Number of distinct steps; step k uses slot k mod period. */
int sgp_schedule_period(const sgp_schedule *s, int64_t *period);
/* Non-zeros of P^(k). */
int sgp_schedule_nnz(const sgp_schedule *s, int64_t k, int64_t *nnz);
/* Copies step k's CSR into HOST arrays rowptr[n+1], col[cap], val[cap]; SGP_ERR_ARG if cap < nnz. */
int sgp_schedule_get(const sgp_schedule *s, int64_t k, int32_t *rowptr, int32_t *col, float *val,
                     int64_t cap, int64_t *nnz);

/* ---------------------------------------------------------------------------------------------
 * Handle: compiled schedule uploaded to the device, the ring of delayed messages (tau > 0) and a
 * few words of launch scratch.  Problem statement: Eq. 1 (n nodes, parameters in R^d).
 * ------------------------------------------------------------------------------------------- */
typedef struct sgp_handle sgp_handle;

#define SGP_FLAG_NONE   0u
#define SGP_FLAG_BIASED 1u    /* Sec. 6.1 / Table 4 "biased OSGP" ablation: z = x, the push-sum weight is mixed and
                                 kept in W but left out of the de-bias */

/*
 * sgp_create: n nodes (1..SGP_MAX_NODES), d parameters per node, ld >= d the row pitch in floats of
 * every n x ld array later passed to this handle, graph schedule g (compiled here), tau >= 0 the
 * fixed message delay of Overlap SGP (Alg. 2; tau = 0 is Alg. 1).  For tau > 0 the handle allocates
 * and zeroes a ring of tau slots of n x ld floats plus tau x n weights (virtual nodes start at
 * zero).  Uses the current CUDA device; later calls on the handle must be made with that device current
 * (SGP_ERR_STATE otherwise).  Synchronises.  On error *out is NULL.
 */
int sgp_create(sgp_handle **out, int n, int64_t d, int64_t ld, const sgp_graph_desc *g, int tau,
               unsigned flags);
/* Frees everything the handle owns.  Synchronises the device.  NULL is accepted. */
int sgp_destroy(sgp_handle *h);
/*
 * sgp_set_graph: replaces the handle's graph schedule (same n) from now on -- the hybrid schemes of
 * Sec. 6.1 / Table 3 (AllReduce-like complete graph or two-peer graph for the first epochs, one-peer
 * graph afterwards).  State, momentum and the delay ring are untouched: messages already in transit
 * are still delivered.  Step k of later calls uses slot k mod (new period).  Synchronises the device.
 * On error the handle keeps its current schedule.
 */
int sgp_set_graph(sgp_handle *h, const sgp_graph_desc *g);
/* The handle's compiled schedule (owned by the handle; valid until sgp_destroy or sgp_set_graph). */
int sgp_get_schedule(const sgp_handle *h, const sgp_schedule **s);

/*
 * sgp_step: one whole SGP iteration k for all n nodes, in ONE pass over HBM (Alg. 1 lines 4-8 with
 * the update of Alg. 3 lines 4-5; Alg. 2 for tau > 0):
 *     g~  = G + weight_decay * X
 *     momentum != 0:  M <- momentum*M + g~ ;  s = momentum*M + g~ (nesterov) or M (otherwise)
 *     momentum == 0:  s = g~                          (d_M may be NULL and is not touched)
 *     h   = X - lr * s
 *     tau == 0:  X_i <- sum_j p_ij h_j ,  W_i <- sum_j p_ij W_j           (CSR order, fp32 FMA)
 *     tau  > 0:  X_i <- p_ii h_i + ring[k mod tau]_i ; ring[k mod tau]_i <- sum_{j != i} p_ij h_j
 *                (same for W): a message sent at step k is consumed by step k + tau
 *     Z_i <- X_i * (1 / W_i)          if d_Z != NULL  (reciprocal rounded once per node)
 * When every row of P^(k) is the same (complete graph) and tau == 0 the mix is formed once per column as
 * a sum of a few interleaved partial sums and shared by all receivers.
 * X, W, M are updated in place; G is only read; Z is only written.  All arrays n x ld fp32 device
 * memory except W (n floats).  Arrays must not overlap.  If every pointer is 16-byte aligned and
 * ld is a multiple of 4 the 128-bit path runs.  Otherwise, if all arrays sit at the same distance from a 16-byte
 * boundary (a dense pitch ld = d with d not a multiple of 4), a kernel that cuts every row at its own 16-byte
 * boundaries runs at about 0.7 of the copy bandwidth; anything else takes a scalar path at about 0.4.  Same results
 * in every case; padding ld is the better answer.
 * k >= 0 selects the schedule slot k mod period and the ring slot k mod tau; for tau > 0 the caller
 * must present k = 0, 1, 2, ... in order.  Asynchronous on `stream`; calls on the same handle must
 * be stream-ordered with respect to each other.
 */
int sgp_step(sgp_handle *h, float *d_X, float *d_W, float *d_M, const float *d_G, float *d_Z,
             int64_t k, float lr, float momentum, float weight_decay, int nesterov, void *stream);

/*
 * sgp_step_adam: the same iteration with the Adam preconditioner in place of the momentum update
 * (Sec. 6.2 and App. C.1: SGP combined with Adam for the Transformer runs; the paper prints no listing,
 * so the update is the standard bias-corrected Adam applied to the numerator with the gradient taken
 * at Z, moments local to each node and never mixed):
 *     g~ = G + weight_decay * X
 *     M1 <- beta1*M1 + (1-beta1) g~ ;  M2 <- beta2*M2 + (1-beta2) g~^2
 *     h  = X - lr/(1-beta1^t) * M1 / ( sqrt(M2)/sqrt(1-beta2^t) + eps )
 * followed by the mix, weight update and de-bias of sgp_step (any tau).  t >= 1 is the 1-based count
 * of Adam steps taken so far including this one; k >= 0 selects the schedule and ring slots.
 * M1, M2 are n x ld fp32 device arrays updated in place (start at zero).  32 bytes of HBM traffic per
 * node-parameter with Z written.
 */
int sgp_step_adam(sgp_handle *h, float *d_X, float *d_W, float *d_M1, float *d_M2, const float *d_G, float *d_Z,
                  int64_t k, int64_t t, float lr, float beta1, float beta2, float eps, float weight_decay,
                  void *stream);

/* sgp_debias: Z_i = X_i * (1 / W_i) for all nodes (Alg. 1 line 8), one pass.  X may equal Z. */
int sgp_debias(sgp_handle *h, const float *d_X, const float *d_W, float *d_Z, void *stream);

/*
 * sgp_step_host: the same iteration for callers whose gradients and parameters live in HOST memory.
 * h_G (read) and h_Z (written, may be NULL) are n x ld host arrays, ideally page-locked; X, W, M stay
 * resident on the device; d_G and d_Z are device staging arrays of n x ld floats supplied by the
 * caller.  The columns are cut into chunks; chunk c's host->device copy, its fused step and its
 * device->host copy overlap with the neighbouring chunks on the handle's three internal streams.
 * Work the caller already enqueued on `stream` is waited for on the device (an event, no host
 * synchronisation on entry).  Returns after everything has completed (synchronises the internal streams).
 * chunk_cols <= 0 picks a default (about 64 MB of gradient per chunk, with smaller chunks at both ends so that
 * the pipeline fills and drains quickly); a positive value cuts the columns into equal chunks of that width.
 */
int sgp_step_host(sgp_handle *h, float *d_X, float *d_W, float *d_M, const float *h_G, float *h_Z,
                  float *d_G, float *d_Z, int64_t k, float lr, float momentum, float weight_decay,
                  int nesterov, int64_t chunk_cols, void *stream);

/* sgp_step_adam_host: the Adam iteration of sgp_step_adam with gradients and de-biased parameters in HOST memory,
 * pipelined like sgp_step_host (Sec. 6.2 / App. C.1 optimiser; same chunking, streams and synchronisation). */
int sgp_step_adam_host(sgp_handle *h, float *d_X, float *d_W, float *d_M1, float *d_M2, const float *h_G, float *h_Z,
                       float *d_G, float *d_Z, int64_t k, int64_t t, float lr, float beta1, float beta2, float eps,
                       float weight_decay, int64_t chunk_cols, void *stream);

/* Zeroes the delay ring (messages in transit are dropped: use only to restart a run). */
int sgp_reset(sgp_handle *h, void *stream);
/* Checkpointing of the in-transit messages: d_ring_x is tau*n*ld floats, d_ring_w is tau*n floats
 * (device memory), slot-major.  SGP_ERR_STATE if tau == 0. */
int sgp_ring_export(sgp_handle *h, float *d_ring_x, float *d_ring_w, void *stream);
int sgp_ring_import(sgp_handle *h, const float *d_ring_x, const float *d_ring_w, void *stream);

/*
 * sgp_colsum: per-column sums in fp64, d_out[c] = sum_i A[i, c] for the n x ld device array A (X, G, M, ...),
 * plus, if include_ring != 0, every entry of the handle's delay ring in that column (the messages in transit:
 * the virtual nodes of the delay model).  d_out is d doubles of DEVICE memory.  Asynchronous on `stream`.
 * Column-stochastic mixing (Sec. 2: every column of P sums to one) conserves exactly these sums, so a caller can
 * form the expected sums of the next state from sums of the current arrays -- e.g. for momentum SGD
 *     colsum(X') + ring' = colsum(X) + ring - lr * (momentum * colsum(M') + colsum(G) + wd * colsum(X))   (Nesterov)
 * -- and hand them to sgp_check.
 */
int sgp_colsum(sgp_handle *h, const float *d_A, int include_ring, double *d_out, void *stream);

/*
 * sgp_check: invariants of column-stochastic mixing (Sec. 2; delay model: mass in transit counts).
 * One pass over X and the ring; one thread per column, fp64 accumulation, warp-shuffle reductions.
 * d_colsum_ref (DEVICE, d doubles, may be NULL): the expected per-column sums of X plus ring (see sgp_colsum).
 * Writes to HOST h_stats[8]:
 *   [0] sum_i W_i + sum of the ring weights (should equal n)      [1] min_i W_i (NaN reported as -1)
 *   [2] number of non-finite entries of X and the ring            [3] sum over all entries of X and the ring
 *   [4] max_c |colsum_c - ref_c|                                  [5] max_c |colsum_c - ref_c| / max(sum_i |x_ic|, |ref_c|)
 *   [6] | [0] - n |                                               [7] the device status word after the check
 * ([4], [5] are 0 without a reference).  The check ORs SGP_STATUS_NONFINITE / ZERO_WEIGHT / WEIGHT_SUM (drift above
 * 1e-4 n) / COLUMN_SUM (relative drift above 1e-5) into the device status word.  Returns, after filling h_stats:
 * SGP_ERR_ZERO_WEIGHT if a weight is <= 0 or NaN, else SGP_ERR_DEVICE if a kernel of this handle ever gave up a
 * bounded wait, else SGP_ERR_INVARIANT if any of the three invariants failed, else SGP_OK.  Synchronises.
 * The weight sum is conserved only to fp32 rounding: weights such as 1/3 make the columns of P sum to 1 within an ulp,
 * and the sum walks away from n by about 4e-5 n per 4000 steps on random digraphs (measured at n = 256), so a run of
 * 1e4 steps and more (n = 256 crosses 1e-4 n after about 10,000 steps) should read [6] against its own history
 * rather than against the fixed bound; the per-step bracket of "check_steps" compares consecutive sums instead.
 */
int sgp_check(sgp_handle *h, const float *d_X, const float *d_W, const double *d_colsum_ref, double *h_stats,
              void *stream);

/*
 * sgp_get_diagnostics: the diagnostics accumulated by the most recent step taken with option "diagnostics" = 1,
 * computed inside the fused pass from the tile already on chip (no extra HBM traffic for tau <= 1; tau - 1 extra
 * ring reads per element otherwise):
 *   h_param_dev[i] = || h_i - (1/n) sum_j h_j ||_2,  h = x^(k+1/2): the parameter deviation of Sec. 6.1 / Fig. 2,
 *                    taken after the gradient step and before the mix;
 *   h_consensus[i] = || z_i^(k+1) - xbar^(k+1) ||_2 with xbar = (1/n) (sum_j x_j + everything in transit): the
 *                    distance bounded by the consensus lemma of the supplement (definition of xbar after Eq. 4).
 * Either HOST array (n doubles) may be NULL.  h_summary (HOST, 6 doubles, may be NULL) receives mean, min, max
 * over nodes of the parameter deviation, then of the consensus distance (the figure plots mean and min..max).
 * Squares are accumulated in fp32 per warp group, fp64 per CTA and across CTAs.  SGP_ERR_STATE if no such step
 * was taken.  Synchronises.
 */
int sgp_get_diagnostics(sgp_handle *h, double *h_param_dev, double *h_consensus, double *h_summary, void *stream);

/*
 * sgp_param_deviation: the parameter-deviation diagnostic of Sec. 6.1 / Fig. 2.  For an n x ld device
 * array A (X, Z or any other per-node array of this handle's shape) writes to HOST h_dev[n] the
 * Euclidean distance of every node's row from the node-wise average row,
 *     h_dev[i] = || A_i - (1/n) sum_j A_j ||_2 ;
 * the figure plots the mean with the min..max band of these n numbers.  One read of A (4 bytes per
 * element); squared differences are accumulated in fp32 per CTA and in fp64 across CTAs.  Synchronises.
 */
int sgp_param_deviation(sgp_handle *h, const float *d_A, double *h_dev, void *stream);

/*
 * Tuning knobs for experiments (defaults are chosen per problem shape):
 *   "variant"      0 = automatic, 1 = register-staged kernel, 2 = TMA pipelined kernel fed by 2-D tensor
 *                  maps, 3 = the same kernel fed by one bulk copy per row segment (no tensor maps), 4 = the
 *                  thread-block-cluster kernel (a cluster of CTAs shares a tile through distributed shared memory)
 *                  -- measured slower than variant 1 at every shape tried, never chosen automatically
 *                  5 = the peeled kernel that the automatic choice takes for rows off the 16-byte grid (each row is
 *                  cut at its own 16-byte boundaries; with aligned rows it runs too, a little slower than variant 1)
 *   "cluster"      CTAs per cluster of variant 4: 0 = 2, 1 = do not use clusters, 2 or 4
 *   "tile_cols"    columns per tile (multiple of 4; 0 = automatic)
 *   "ctas_per_sm"  persistent CTAs per SM (0 = automatic)
 *   "stages"       shared-memory stages of the bulk-copy pipeline (0 = automatic, at most 8)
 *   "single_buffer" register-staged kernel: 0 = automatic (from n and the tile width), 1 = one exchange tile and two barriers
 *                  per tile, 2 = two exchange tiles and one barrier
 *   "lockstep"     register-staged kernel: 2 or 4 = launch it as thread-block clusters of that many CTAs that take
 *                  neighbouring tiles and meet at a cluster barrier before each tile (they share no data; it only
 *                  aligns their memory traffic in time), 1 = independent CTAs, 0 = automatic (clusters when rows do
 *                  not start on 128-byte boundaries, where they win back about 4 % of the bandwidth, and for
 *                  tau >= 1 at 1 KB row segments).  Results do not depend on it, bit for bit.
 *   "wait_limit_ms" bound of every in-kernel wait of the pipelined kernel (0 = 2000 ms); a wait that runs out
 *                  sets the device status word (sgp_device_status) and the CTA leaves: nothing hangs
 *   "inject_stall" test hook, 0/1: one CTA of the pipelined kernel never requests its first tile, so that
 *                  the bounded wait and the status word can be exercised (that step's results are invalid)
 *   "l2_hint"      L2 evict-first policy on the pipeline's bulk copies: 0 = automatic (gradients only),
 *                  1 = every array, 2 = none, 3 = gradients only, 4 = every array but the gradients
 *   "send_period"  s >= 1 (default 1): nodes transmit only on steps with k mod s == 0 and keep their whole half step
 *                  (identity mixing matrix) otherwise -- Alg. 2 lines 5-12 taken literally with s = tau; the c-th
 *                  transmission uses schedule slot c mod period; messages still arrive tau steps after they were sent
 *   "diagnostics"  0/1: accumulate the parameter deviation and the consensus distance inside every step
 *                  (sgp_get_diagnostics reads the latest)
 *   "check_steps"  0/1, debug: every step is bracketed by an expected-column-sum pre-pass and a column-sum check
 *                  (sum_i x_i' plus ring against sum_i h_i plus ring, Sec. 2); a drift sets SGP_STATUS_COLUMN_SUM in
 *                  the device status word, and a weight sum (weights in transit included) that differs from the one
 *                  taken just before the step by more than 1e-5 n sets SGP_STATUS_WEIGHT_SUM (one step keeps the sum
 *                  to a few roundings).  Costs about two extra passes over the arrays and 8 d bytes of device
 *                  memory, allocated when the option is switched on (SGP_ERR_ALLOC if that fails)
 * Read-only through sgp_get_option: "last_variant", "last_grid", "last_smem", "last_tile_cols", "last_lockstep" describe
 * the most recent step launch of the handle (which kernel ran, CTAs, dynamic shared memory, tile width);
 * "launches" counts the step kernels the handle has launched so far.
 * Unknown keys or unsupported values return SGP_ERR_ARG and change nothing.
 */
int sgp_set_option(sgp_handle *h, const char *key, int64_t value);
int sgp_get_option(const sgp_handle *h, const char *key, int64_t *value);

/*
 * sgp_step_static: the tau = 0 fused step of sgp_step for callers that cannot allocate device memory.
 * (The paper has no counterpart: this entry point exists for deployment reasons only.)
 *
 * Who needs it: a process whose device memory was handed, whole, to a framework's pool at start-up; a
 * latency-critical loop that cannot afford the device-wide synchronisation an allocation implies; a
 * plug-in running under a memory-accounting wrapper.  sgp_create allocates, so these callers use no
 * handle.  This call performs no cudaMalloc/cudaFree and calls no allocating library routine: the
 * step's in-neighbour table and its two launch words live in one file-scope device array inside the
 * library image (about 40 KB, held by every GPU that loads the library until the process exits).
 *
 * The mixing matrix of the step is passed as HOST arrays in the CSR form sgp_schedule_get produces
 * (h_rowptr[n+1], h_col[nnz], h_val[nnz]; the host-only schedule compiler needs no GPU).  Limits:
 * n <= SGP_MAX_NODES and nnz <= SGP_STATIC_MAX_NNZ, otherwise SGP_ERR_ARG ("use a handle"); a table
 * whose row pointers or column indices are inconsistent, whose senders are not ascending inside a row, that
 * lacks a self-loop, or whose columns do not sum to one (the schedule compiler's rule) returns SGP_ERR_GRAPH.
 * X, W, M are updated
 * in place, G is read, Z (may be NULL) is written, exactly as by sgp_step; M may be NULL when
 * momentum == 0.  Asynchronous on `stream`.
 *
 * Set-up: the first call made with a given device current resolves the device address of the static
 * array (cudaGetSymbolAddress) and caches it for that device; make that first call outside any stream
 * capture.  A call whose `stream` is being captured is refused with SGP_ERR_STATE: the table upload reads the
 * caller's host arrays when it executes, and those are only promised to live for the duration of the call.
 * Sharing: all calls on a device use the same array, and it keeps the last call's
 * contents; every call rewrites the table and clears the launch words in stream order, so calls
 * issued to ONE stream are safe back to back, while calls that may overlap on the GPU (different
 * streams without a dependency) race and must not be made.
 */
#define SGP_STATIC_MAX_NNZ 4096
int sgp_step_static(int n, int64_t d, int64_t ld, const int32_t *h_rowptr, const int32_t *h_col,
                    const float *h_val, int64_t nnz, float *d_X, float *d_W, float *d_M, const float *d_G,
                    float *d_Z, float lr, float momentum, float weight_decay, int nesterov, void *stream);

/* ---------------------------------------------------------------------------------------------
 * One node per GPU (App. C "Implementation Details": every node sends (p x, p w) to its out-neighbours and adds
 * what it receives; Sec. 3 "Overlapping communication and computation", Alg. 2).  Rank r of `world` = n nodes
 * holds ONE row of every array: x, m, g, z are d floats, w is one float, all DEVICE memory of the caller.
 * The step is split where data crosses between nodes:
 *     update : h = x - lr * s, written UNWEIGHTED with w into a message slot in this GPU's memory (the "send")
 *     mix    : x' = sum_j p_ij h_j, w' = sum_j p_ij w_j, z = x' / w', reading every in-neighbour's slot directly
 *              from that GPU's memory with plain loads over NVLink (peer pointers): pull and mix are one kernel;
 *              the receiver applies p_ij, so all out-neighbours of a node read the same slot
 *     tau >= 1 : the messages consumed at step k were published at step k - tau, so update + pull + mix are ONE
 *              kernel per step (sgp_rank_step_overlap) and the exchange never waits.
 * Results are bit-identical to sgp_step on the stacked n x d arrays (same CSR order, same FMA chain); the one
 * exception is sgp_step's shortcut for steps whose rows of P are all alike with tau == 0 (complete graph), which sums
 * interleaved partial sums: there the two agree to rounding, not bit for bit.
 *
 * Synchronisation is the caller's (one barrier per step across the ranks, e.g. an all-reduce of one element on the
 * step's stream): tau == 0: update, BARRIER, mix; tau >= 1: step_overlap, BARRIER.  No kernel of this library
 * waits on another GPU.  A rank keeps tau + 2 message slots: a slot is rewritten tau + 2 steps after it was
 * published, when every reader has passed at least one barrier since its read.
 * Not supported here: send_period, in-degree above SGP_RANK_MAX_SOURCES (SGP_ERR_ARG; the complete graph
 * is what an all-reduce is for).
 * ------------------------------------------------------------------------------------------- */
typedef struct sgp_rank sgp_rank;
#define SGP_RANK_MAX_SOURCES 32
#define SGP_IPC_HANDLE_BYTES 64

/* What rank `rank` does at step k (HOST only, needs no GPU): which slot it publishes into, which slot of its
 * in-neighbours it reads, its own weight p_ii^(k), and the in-neighbours with the weights p_ij it applies, in the
 * order of the sum.  tau == 0: the list is row `rank` of P^(k), self included at self_pos, read_slot == write_slot.
 * tau >= 1: the list is row `rank` of P^(k - tau) without the diagonal (empty while k < tau: nothing has
 * arrived yet), self_pos = -1, and the node's own half step enters with self_weight. */
typedef struct sgp_rank_plan_t {
  int32_t write_slot, read_slot;
  float   self_weight;
  int32_t self_pos;
  int32_t count;
  int32_t sender[SGP_RANK_MAX_SOURCES];
  float   weight[SGP_RANK_MAX_SOURCES];
} sgp_rank_plan_t;
int sgp_rank_plan(const sgp_schedule *s, int rank, int64_t k, int tau, sgp_rank_plan_t *out);
/* The same with a send period s >= 1 (Alg. 2 line 5; the stacked path's "send_period" option): nodes transmit only on
 * steps k with k mod s == 0, and the c-th transmission (k = c s) uses P^(c).  On every other step the matrix is the
 * identity: self_weight = 1 and, for tau == 0, the list holds the node itself alone; for tau >= 1 the list is empty
 * unless step k - tau was a transmission, whose off-diagonal row then arrives.  send_period == 1 is sgp_rank_plan. */
int sgp_rank_plan_period(const sgp_schedule *s, int rank, int64_t k, int tau, int64_t send_period, sgp_rank_plan_t *out);

/* Creates rank `rank` of `world` on the current device: compiles the schedule for n = world nodes and allocates
 * and zeroes (tau + 2) message slots of d (+ padding) floats.  Synchronises. */
int sgp_rank_create(sgp_rank **out, int rank, int world, int64_t d, const sgp_graph_desc *g, int tau, unsigned flags);
int sgp_rank_destroy(sgp_rank *r);
int sgp_rank_get_schedule(const sgp_rank *r, const sgp_schedule **s);
/* The rank's message slots: one device allocation of `bytes` bytes.  Other ranks need its address in THEIR
 * process: the same pointer inside one process, or sgp_ipc_export here + sgp_ipc_open there.  The block is plain
 * device memory holding every message still in transit: a checkpoint copies its `bytes` out (with x, u, w) and a
 * restart copies them back into the block of a rank created with the same arguments before its next step. */
int sgp_rank_message_block(sgp_rank *r, void **d_block, size_t *bytes);
/* d_peer_blocks[j] (HOST array of `world` device pointers valid in this process; entry [rank] is ignored, entries
 * of ranks this node never receives from may be NULL): where rank j's message block is mapped. */
int sgp_rank_set_peers(sgp_rank *r, void *const *d_peer_blocks);
/* Send period of this rank's steps (default 1, at most 2^20); every rank of a run must set the same value before
 * the first step. */
int sgp_rank_set_send_period(sgp_rank *r, int64_t send_period);
/* tau == 0, first half: publishes (h, w) of step k; m updated in place; x untouched.  Asynchronous. */
int sgp_rank_update(sgp_rank *r, const float *d_x, float *d_w, float *d_m, const float *d_g, int64_t k, float lr,
                    float momentum, float weight_decay, int nesterov, void *stream);
/* tau == 0, second half, after every in-neighbour's update of step k is complete: pull + mix + de-bias; writes x,
 * w, z (d_z may be NULL).  SGP_ERR_STATE if tau != 0 or a needed peer block was never set.  Asynchronous. */
int sgp_rank_mix(sgp_rank *r, float *d_x, float *d_w, float *d_z, int64_t k, void *stream);
/* tau >= 1: the whole step k in one kernel (Alg. 2).  Steps must be presented in order.  SGP_ERR_STATE if
 * tau == 0.  Asynchronous. */
int sgp_rank_step_overlap(sgp_rank *r, float *d_x, float *d_w, float *d_m, const float *d_g, float *d_z, int64_t k,
                          float lr, float momentum, float weight_decay, int nesterov, void *stream);
/* The same two calls with the Adam preconditioner (Sec. 6.2 / App. C.1; arguments as sgp_step_adam: t >= 1 counts
 * the Adam steps including this one; m1, m2 are this node's moment rows, never sent). */
int sgp_rank_update_adam(sgp_rank *r, const float *d_x, float *d_w, float *d_m1, float *d_m2, const float *d_g, int64_t k,
                         int64_t t, float lr, float beta1, float beta2, float eps, float weight_decay, void *stream);
int sgp_rank_step_overlap_adam(sgp_rank *r, float *d_x, float *d_w, float *d_m1, float *d_m2, const float *d_g, float *d_z,
                               int64_t k, int64_t t, float lr, float beta1, float beta2, float eps, float weight_decay,
                               void *stream);
/* SGP_STATUS_ZERO_WEIGHT is the only bit this mode sets.  Synchronises. */
int sgp_rank_device_status(sgp_rank *r, unsigned *status);
/* Thin wrappers of the CUDA IPC calls for callers without a CUDA binding: `handle` is SGP_IPC_HANDLE_BYTES bytes of
 * HOST memory to ship to the other process by any means; sgp_ipc_open maps the exporter's allocation into this
 * process (peer access is enabled as needed) and sgp_ipc_close unmaps it. */
int sgp_ipc_export(const void *d_ptr, unsigned char *handle);
int sgp_ipc_open(const unsigned char *handle, void **d_ptr);
int sgp_ipc_close(void *d_ptr);

/* Reads the handle's device status word (SGP_STATUS_* bits; 0 = nothing ever went wrong).  Once a wait bit or
 * the zero-weight bit has been seen by a synchronising call (this one, sgp_check, sgp_step_host), later
 * sgp_step / sgp_step_adam calls return SGP_ERR_DEVICE / SGP_ERR_ZERO_WEIGHT until sgp_reset, which clears the
 * word.  Synchronises. */
int sgp_device_status(sgp_handle *h, unsigned *status);
/* cudaError_t value latched by the last call that returned SGP_ERR_CUDA on this handle (0 if none). */
int sgp_last_cuda_error(const sgp_handle *h);
const char *sgp_strerror(int code);
/* Library version as major*10000 + minor*100 + patch. */
int sgp_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SGP_H_ */
