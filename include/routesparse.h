/*
 * routesparse.h -- C ABI of the routed structured-sparse causal prefill attention path (RouteSparse).
 *
 * One attention layer at a time, on one GPU (sm_100a).  The calls follow the paper's per-layer procedure
 * (Section 3.4, the six-step table): probe -> candidate indices, coverage, uncertainty -> routing under the
 * layer budget with fallback -> one sparse attention launch for all heads -> certificate.
 *
 * Conventions (all entry points)
 *   - Return value: RS_OK or a negative rs_status.  Nothing is thrown; nothing is printed.
 *   - Every tensor pointer is a DEVICE pointer owned by the caller unless the comment says "host".
 *     The library allocates no device memory: scratch comes from the caller's workspace
 *     (rs_workspace_bytes), which must be 256-byte aligned.
 *   - Every call only enqueues work on `stream` (a cudaStream_t passed as void*); it neither synchronises nor
 *     copies to the host.  Conditions only knowable on the device (a bounded wait that expired, an
 *     infeasible budget) are written to `status` (device int32[RS_STATUS_WORDS], may be NULL).
 *   - Layouts are contiguous, row-major: Q[n_q_heads][n_keys][d], K and V [n_kv_heads][n_keys][d], bf16,
 *     d = 128.  Query head h reads KV head h / (n_q_heads / n_kv_heads).
 *   - A segment s is the query range [seg_bounds[s], seg_bounds[s+1]) attending keys [0, seg_bounds[s+1]).
 *     Bounds are multiples of 64; seg_bounds[0] = 0; seg_bounds[n_segments] = n_keys.  Items are
 *     (segment, head) pairs, item = s * n_q_heads + h.
 *   - Probe rows: the last 64 query rows of a segment, in four groups of 16 consecutive rows.
 */
#ifndef ROUTESPARSE_H_
#define ROUTESPARSE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RS_BLOCK 64          /* block edge of block-sparse blocks and of block diagonals */
#define RS_PROBE_ROWS 64
#define RS_PROBE_GROUPS 4
#define RS_HEAD_DIM 128
#define RS_STATUS_WORDS 8    /* [0] first error code, [1] where, [2..] kernel specific */
#define RS_MAX_KEYS 262144
#define RS_MAX_CANDIDATES 32

typedef enum {
  RS_OK = 0,
  RS_ERR_INVALID_ARG = -1,
  RS_ERR_UNSUPPORTED_SHAPE = -2,
  RS_ERR_WORKSPACE_TOO_SMALL = -3,
  RS_ERR_CUDA = -4,
  RS_ERR_UNSUPPORTED_DEVICE = -5,
  RS_ERR_TIMEOUT = -6,
  RS_ERR_NOALLOC_TOO_LARGE = -7
} rs_status;

/* Pattern library of Section 3.1. */
typedef enum { RS_DENSE = 0, RS_A_SHAPE = 1, RS_VERTICAL_SLASH = 2, RS_BLOCK_SPARSE = 3 } rs_pattern;

/* One (pattern, budget) pair.  Budgets "in units that match the kernel" (Section 3.1):
 *   A-shape: b0 = sink tokens, b1 = local window width (tokens, diagonal included)
 *   vertical-slash: b0 = k_v columns, b1 = k_s slash offsets (offset 0 is always kept and counted)
 *   block-sparse: b0 = k_b key blocks per query block (the diagonal block is always kept and counted)
 *   dense: none.
 * Within a family the library lists candidates by increasing budget ("expand" = next of the family). */
typedef struct { int32_t pattern, b0, b1, flags; } rs_candidate;

typedef struct {
  int32_t n_q_heads, n_kv_heads, head_dim, n_keys;
  int32_t n_segments;
  const int32_t* seg_bounds;   /* HOST array, n_segments + 1 entries */
} rs_problem;

/* Index storage (device arrays owned by the caller).  Two uses:
 *   evaluation  (choice == NULL): VS slot = item * n_cand + c;  bs_blk holds, per slot, only the list of the
 *                segment's last query block: bs_rows = n_items * n_cand.
 *   materialised (choice != NULL): VS slot = item;  bs_blk is indexed by (head, global query block):
 *                bs_rows = n_q_heads * n_keys / 64.
 * Lists are ascending.  Unused tail entries are unspecified.
 * rs_sparse_prefill_attn accepts the vertical-slash arrays in either layout (it tells them apart by n_vs_slots ==
 * n_items * n_cand), so a caller that has evaluated every candidate need not build the chosen lists again: it passes
 * n_vs_slots = 0 to the materialising rs_build_indices call (block-sparse rows only) and hands the attention call the
 * evaluation's vertical-slash arrays together with the materialised block-sparse arrays. */
typedef struct {
  int32_t n_vs_slots, kv_cap, ks_cap, nd_cap;   /* capacities per slot (>= largest budget / n_keys/64) */
  int32_t bs_rows, kb_cap;
  int32_t* vs_cols;    /* [n_vs_slots][kv_cap]  vertical key indices */
  int32_t* vs_offs;    /* [n_vs_slots][ks_cap]  slash offsets */
  int32_t* vs_diag;    /* [n_vs_slots][nd_cap]  block-diagonal deltas D */
  int32_t* vs_count;   /* [n_vs_slots][4]       n_cols, n_offs, n_diag, 0 */
  int32_t* bs_blk;     /* [bs_rows][kb_cap]     selected key blocks */
  int32_t* bs_count;   /* [bs_rows] */
} rs_index_set;

/* Per (item, candidate): fixed-point covered probe mass per probe group (unit 2^-32; m_hat_g = cov_fx[g] /
 * (16 * 2^32)) and the exact number of selected causal query-key pairs. Dense: cov_fx unused. */
typedef struct { uint64_t cov_fx[RS_PROBE_GROUPS]; uint64_t pairs; } rs_cand_stats;

typedef enum { RS_CERT_ABS = 0, RS_CERT_REL = 1 } rs_cert_mode;

typedef struct {
  int64_t budget;          /* T_l of Eq. 8, same integer unit as cost */
  int64_t t_probe;         /* t_probe of Eq. 8 */
  double alpha;            /* weight of u in Eq. 4 */
  double delta_q;          /* m_low = max(0, m_hat - delta_q) */
  double cert_max;         /* fallback fires while certificate > cert_max */
  int32_t use_cert;        /* 0: no fallback step */
  int32_t cert_mode;       /* rs_cert_mode: REL 2(1-m_low), ABS 2(1-m_low) * V_max */
  int32_t expand_first;    /* 1: next larger budget of the family before dense */
  int32_t rescue_any;      /* 1 = when the family has no larger budget, take the cheapest sparse candidate of any
                              family whose certificate passes before giving up and going dense */
  const int32_t* forced_dense;  /* device int32[n_items], non-zero = force dense last; may be NULL */
  const int32_t* fixed_choice;  /* device int32[n_items]; when set, bypasses solve and fallback; may be NULL */
  const double* e;         /* device double[n_items][n_cand]: calibrated error predictor e of Eq. 4 (rs_regressor_eval);
                              NULL or beta == 0: the training-free router */
  double beta;             /* weight of e in Eq. 4 */
  int32_t backfill;        /* 1: after the greedy solve, spend what is left of the budget on the substitutions with
                              the largest risk decrease per unit of added cost that still fit (before the fallback) */
  int32_t global_pattern;  /* 1: the layer-level comparison router of Section 4 (baselines): every item takes the
                              same candidate, the feasible one with the smallest summed risk (ties: cheaper, lower
                              index); the greedy solve and the back-fill are skipped, the fallback still runs */
  const uint64_t* cov_mix; /* device uint64[n_items][n_cand][4] from rs_mixture_coverage, or NULL.  When set, u of Eq. 4
                              is the disagreement among the row subsets of the query mixture, max_b m_b - min_b m_b with
                              m_b = cov_mix[..][b] / (mix_rows[b] * 2^32), instead of the spread over the four groups of
                              the last 64 rows */
  int32_t mix_rows[4];     /* rows per subset (0 = subset unused) */
} rs_route_params;

/* total_cost and total_risk are those of the final routes (t_probe included in the cost).  feasible is the outcome of
 * the budgeted solve of Eq. 6-8 alone (0: even the cheapest candidates exceed the budget); the fallback walk and the
 * forced-dense set run afterwards and may push total_cost above the budget again (Section 3.4, step 5), which a caller
 * sees by comparing total_cost with the budget it passed. */
typedef struct { int64_t total_cost; double total_risk; int32_t n_fallback; int32_t feasible; } rs_route_report;

const char* rs_error_string(int code);
int rs_version(void);

/* Streams and graphs.  Every call below only enqueues work on the caller's stream; rs_probe and rs_build_indices also
 * use one internal side stream per device for kernels that do not depend on each other, forked from and joined back
 * into the caller's stream with events, so the caller still sees one ordered piece of work and the calls can be
 * captured into a CUDA graph.  The first call of an entry point on a device sets kernel attributes and creates that
 * side stream: make it outside any capture.  Calls from several host threads on one device are serialised while they
 * hold the side stream. */

/* Bytes of scratch that any hot-path call below needs for this problem and library (host computation). */
int rs_workspace_bytes(const rs_problem* p, const rs_candidate* lib, int n_cand, size_t* bytes);

/* Shared attention probe, Eq. 3 (Section 3.2) in the last-64-query form, for every (segment, head):
 * exact softmax rows of the last 64 queries over all causal keys, reduced to
 *   vert  [n_seg][n_q_heads][4][n_keys]  column mass per probe group          (fp32, 0 beyond the segment end)
 *   slash [n_seg][n_q_heads][4][n_keys]  diagonal mass per offset i - j        (fp32)
 *   lse_probe [n_q_heads][n_seg][64]     log-sum-exp of each probe row         (fp32; the layout rs_certificate
 *                                        takes as lse_full for rows = the segments' last 64 rows)
 * plus the pooled signals of the coarse block candidates and the value norms of Eq. 5:
 *   qpool [n_q_heads][n_keys/64][d], kpool [n_kv_heads][n_keys/64][d]  64-row means (fp32)
 *   vmax  [n_seg][n_kv_heads]   max_j ||v_j||_2 over j < segment end             (fp32)
 * vert and slash are fully overwritten.  descr (may be NULL): [n_seg][n_q_heads][2], two of the descriptors of
 * Section 3.2 on the exact probe rows: entropy (mean over the 64 rows of -sum_j p ln p, in nats) and local-band
 * concentration (mean over the rows of the mass of keys with i - j < 1024). */
int rs_probe(const rs_problem* p, const void* Q, const void* K, const void* V,
             float* vert, float* slash, float* lse_probe, float* qpool, float* kpool, float* vmax,
             float* descr, int flags, void* ws, size_t ws_bytes, int32_t* status, void* stream);

/* The same probe on the query mixture of Eq. 3 at key resolution ("a deterministic mixture of recent, uniformly
 * spaced, and boundary-adjacent positions", Section 3.2): instead of the last 64 rows, four caller-chosen runs of 16
 * consecutive rows per segment (a diagonal is only visible on consecutive rows, so the mixture is made of runs).
 *   run_starts  HOST int32 [n_seg][4]: first row of each run; 0 <= start and start + 16 <= segment end
 *   vert, slash [n_seg][n_q_heads][4][n_keys]: column mass and diagonal mass of run g (group g), fully overwritten;
 *               slash[..][g][o] = sum over the run's rows i >= o of P[i][i - o]
 *   lse_probe   [n_q_heads][n_seg][64]: log-sum-exp of the 64 rows in run order
 * No pooled means, no value norms (rs_probe provides them).  The paper's "Recent queries only" ablation (Table 3) is
 * rs_probe; with the masses of this call handed to rs_build_indices_ranked the line lists are chosen from the mixture. */
int rs_probe_runs(const rs_problem* p, const void* Q, const void* K, const int32_t* run_starts,
                  float* vert, float* slash, float* lse_probe, void* ws, size_t ws_bytes, int32_t* status, void* stream);

/* The query sets I of Eq. 3 ("a deterministic mixture of recent, uniformly spaced, and boundary-adjacent positions";
 * the paper fixes neither proportions nor spacing, these are this library's choices).  Host functions.
 * rs_mixture_rows: rows [r_recent + r_uniform + r_boundary] (host, out) = the last r_recent rows of the segment
 *   [q0, q1), then r_uniform rows at the midpoints of equal strata of what lies between the other two groups, then
 *   the r_boundary rows right after q0; RS_ERR_UNSUPPORTED_SHAPE when the segment is too short for the groups to be
 *   disjoint.  This is the row set rs_probe_pooled and rs_mixture_coverage are meant to be given.
 * rs_mixture_runs: run_starts [4] (host, out) = first rows of the four 16-row runs rs_probe_runs takes: the run right
 *   after q0, the runs one third and two thirds into the segment (in units of 16 rows), and the last 16 rows. */
int rs_mixture_rows(int q0, int q1, int r_recent, int r_uniform, int r_boundary, int32_t* rows);
int rs_mixture_runs(int q0, int q1, int32_t* run_starts);

/* rs_probe flag: fill only the rows of qpool that candidate evaluation reads (the last query block of every segment)
 * and leave the rest to rs_pool_queries once the routes are known; reading all of Q for the pooled means is the
 * largest single stream of the probe (1 GB at 128K) and only heads routed to block-sparse need it. */
#define RS_PROBE_QPOOL_LAST_ONLY 1

/* 64-row means of Q (the rows of qpool rs_probe left out) for the heads whose routed candidate is block-sparse:
 * the pooled queries of Section 3.1 ("pooled queries and keys score coarse blocks"), which the block-sparse family
 * ranks key blocks with.  choice: device int32[n_items] (NULL: every head).  qpool as for rs_probe. */
int rs_pool_queries(const rs_problem* p, const void* Q, const rs_candidate* lib, int n_cand, const int32_t* choice,
                    float* qpool, int32_t* status, void* stream);

/* Candidate index construction and coverage (Section 3.1, 3.2; step 2 of the procedure table).
 * Ranking keys are the integers sum_g floor(mass_g * 2^32); order is key descending, index ascending.
 * vertical-slash: V = top-k_v columns, S = {0} + top-(k_s-1) offsets, D = {floor(o/64), ceil(o/64)}.
 * block-sparse: per query block the diagonal block plus the top-(k_b-1) pooled scores
 *   (qpool . kpool / sqrt(d); `bscore` [n_items][n_keys/64][n_keys/64], indexed by global query block,
 *   replaces the fused product when not NULL).
 * choice == NULL: evaluate every candidate of every item (lists + stats, see rs_index_set).
 * choice != NULL (device int32[n_items]): materialise only the chosen candidate of each item.
 * Limits: every segment needs at least 64 rows (the probe rows), and with stats != NULL an A-shape candidate whose sink
 * columns and window overlap on the probe rows of some segment (window < segment end and segment end - 64 - window + 1 <
 * sink columns) is refused with RS_ERR_UNSUPPORTED_SHAPE: the joint coverage of the two parts cannot be had from the
 * column and offset masses alone.  Budgets larger than a segment are clamped to what exists. */
int rs_build_indices(const rs_problem* p, const rs_candidate* lib, int n_cand,
                     const float* vert, const float* slash, const float* qpool, const float* kpool,
                     const float* bscore, const int32_t* choice,
                     const rs_index_set* out, rs_cand_stats* stats,
                     void* ws, size_t ws_bytes, int32_t* status, void* stream);

/* rs_build_indices with the vertical columns and slash offsets RANKED by another pair of mass arrays (same shapes):
 * V and S are the top-k of rank_vert / rank_slash (the query mixture of Eq. 3, rs_probe_runs), while coverage, the
 * uncertainty groups and everything else are still measured on vert / slash (the last 64 rows, which the certificate
 * audits).  Section 3.2: the probe's mixture of rows decides which lines are worth keeping. */
int rs_build_indices_ranked(const rs_problem* p, const rs_candidate* lib, int n_cand,
                            const float* vert, const float* slash, const float* rank_vert, const float* rank_slash,
                            const float* qpool, const float* kpool, const float* bscore, const int32_t* choice,
                            const rs_index_set* out, rs_cand_stats* stats,
                            void* ws, size_t ws_bytes, int32_t* status, void* stream);

/* Risk (Eq. 4), greedy substitution for the budgeted routing problem (Eq. 6-8), fallback walk and forced
 * dense (Section 3.4), solved by one thread block on the device.
 * cost: device int64[n_items][n_cand] or NULL (then 4 * d * pairs, i.e. FLOPs of the selected pairs).
 * vmax: [n_seg][n_kv_heads].  choice: device int32[n_items] out.  report: device, may be NULL. */
int rs_route(const rs_problem* p, const rs_candidate* lib, int n_cand,
             const rs_cand_stats* stats, const int64_t* cost, const float* vmax,
             const rs_route_params* params, int32_t* choice, rs_route_report* report,
             int32_t* status, void* stream);

/* Masked attention O~ = softmax(Q K^T / sqrt(d) + C + mask(M)) V (Section 2.1) for every head under its
 * routed pattern, one launch for all heads (Section 3.4, step 6).
 * idx: materialised index set; choice: device int32[n_items].
 * O: [n_q_heads][n_keys][d], bf16 (o_dtype 0) or fp32 (o_dtype 1).
 * lse_sel [n_q_heads][n_keys]: log-sum-exp over the selected keys;  onorm (may be NULL): ||O~_i||_2.
 * counters (may be NULL): device uint64[2], incremented by the 64-key chunks issued and by the work items. */
int rs_sparse_prefill_attn(const rs_problem* p, const void* Q, const void* K, const void* V,
                           const rs_candidate* lib, int n_cand, const rs_index_set* idx, const int32_t* choice,
                           void* O, int o_dtype, float* lse_sel, float* onorm, uint64_t* counters,
                           void* ws, size_t ws_bytes, int32_t* status, void* stream);

/* Dense causal attention, Eq. 1, with the same engine (the denominator of "speed-up over own dense").
 * lse [n_q_heads][n_keys] is the full-row log-sum-exp (the audit input of rs_certificate). */
int rs_dense_prefill_attn(const rs_problem* p, const void* Q, const void* K, const void* V,
                          void* O, int o_dtype, float* lse, float* onorm, uint64_t* counters,
                          void* ws, size_t ws_bytes, int32_t* status, void* stream);

/* Dense causal attention for callers that cannot pass a workspace (the paper has no counterpart: this is a
 * convenience of this library, not a step of the method).  Same computation and outputs as rs_dense_prefill_attn,
 * but the launch's work list lives in a fixed array inside the library image instead of caller scratch, so the call
 * needs no device allocation of any kind.  Meant for callers that cannot allocate where they call from: a plugin
 * that only receives its input and output tensors, code running inside an allocator or memory-pool callback, a
 * serving loop in which cudaMalloc (a device-wide synchronisation) is not allowed.
 *   limit   n_q_heads x (number of 128-row query tiles) <= 16384 (e.g. 32 heads at n = 65536); larger problems
 *           return RS_ERR_NOALLOC_TOO_LARGE and nothing is launched.  The array is 320 KB and every GPU that loads
 *           the library keeps it until the process ends.
 *   set-up  the first call on each device looks up the array's device address (with that device current); make that
 *           first call outside any stream capture.  Later calls on the device do no set-up.
 *   sharing all calls on a device use the same array and it keeps the previous call's contents; each call rewrites
 *           every entry it reads, so nothing needs clearing, but two calls whose kernels overlap on the GPU (different
 *           streams without ordering) race on it.  Calls on one stream are safe.
 * No counters output; status as for the other calls (may be NULL). */
int rs_dense_prefill_attn_noalloc(const rs_problem* p, const void* Q, const void* K, const void* V,
                                  void* O, int o_dtype, float* lse, float* onorm, int32_t* status, void* stream);

/* Error certificate, Eq. 5: for audited rows with both log-sum-exps known,
 *   m_i = min(1, exp(lse_sel_i - lse_full_i)),  cert_i = 2 (1 - m_i) V_max,
 *   tight_i = (1 - m_i) (V_max + onorm_i) (written when onorm and cert_tight are given),
 * and per head: m_head = mean_i m_i, cert_head[h][0] = 2 (1 - max(0, m_head - delta_q)) V_max,
 * cert_head[h][1] = max_i cert_i.
 * lse_sel, onorm: [n_q_heads][n_keys].  rows: device int32[n_rows] query row ids (same for every head);
 * lse_full: [n_q_heads][n_rows].  vmax: [n_kv_heads], any upper bound of the value norms of that KV head
 * (rs_probe's vmax row of the last segment qualifies).
 * Outputs (each may be NULL) m_row, cert_row, cert_tight: [n_q_heads][n_rows]; m_head [n_q_heads];
 * cert_head [n_q_heads][2].
 * A row id outside [0, n_keys) is not read: its outputs are NaN, it is left out of the head-level values, and
 * RS_ERR_INVALID_ARG is written to `status` (device, may be NULL). */
int rs_certificate(int n_q_heads, int n_kv_heads, int n_keys, const float* lse_sel, const float* lse_full,
                   const int32_t* rows, int n_rows, const float* vmax, const float* onorm, float delta_q,
                   float* m_row, float* cert_row, float* cert_tight, float* m_head, float* cert_head,
                   int32_t* status, void* stream);

/* Shared attention probe of Eq. 3 (Section 3.2) in its general form: r sampled query rows per (segment, head) against
 * keys pooled over blocks of width g, S = Q[I] pool_g(K)^T / sqrt(d), soft-maxed over the visible key blocks, and the
 * three descriptors of Section 3.2.  The paper leaves open what this library fixes as follows: a key block is visible
 * to row i when its first key is <= i and is pooled (arithmetic mean) over its visible keys only; the agreement
 * descriptor is 1 - total-variation distance between the mean signatures of the first two row subsets, the signature
 * of a row being its mass re-binned into [key block 0] + [relative block offsets 0..15] + [everything else].
 *   rows        device int32[n_seg][r], row ids inside the segment (r <= 64); the caller chooses the mixture of
 *               recent, uniformly spaced and boundary-adjacent positions
 *   g           pooling width, a divisor of 64
 *   sub_bounds  HOST int32[n_sub + 1], 0 = b_0 < ... < b_n_sub = r: the row subsets (n_sub <= 4)
 *   A           device fp32 [n_seg][n_q_heads][r][n_keys / g] out: probabilities (0 on invisible blocks)
 *   lse         device fp32 [n_seg][n_q_heads][r] out
 *   colmass     device fp32 [n_seg][n_q_heads][n_sub][n_keys / g] out: sum over the subset's rows of A[i][kb]
 *   diagmass    same shape, indexed by relative block offset: sum over the subset's rows of A[i][i / g - delta]
 *   descr       device fp32 [n_seg][n_q_heads][4] out: entropy (mean of H_i / log max(2, visible_i)), local-band
 *               mass (blocks whose first key lies within 1024 of the row), agreement, mean number of visible blocks
 *   scratch     device fp32, rs_probe_pooled_scratch_floats() elements
 * Query heads per KV head must be <= 4.  Errors as for the other calls; nothing is allocated. */
int rs_probe_pooled_scratch_floats(const rs_problem* p, int r, size_t* n_floats);
int rs_probe_pooled(const rs_problem* p, const void* Q, const void* K, const int32_t* rows, int r, int g,
                    const int32_t* sub_bounds, int n_sub, float* A, float* lse, float* colmass, float* diagmass,
                    float* descr, float* scratch, int32_t* status, void* stream);

/* Coverage of every candidate's mask on the rows of the query mixture (Section 3.2), the input of the "disagreement
 * among probe subsets" u of Eq. 4.  A comes from rs_probe_pooled at g = 64 (key blocks = the pattern blocks); the mass of
 * a key block is split evenly over its visible keys, so row i of candidate c collects
 *   sum over key blocks kb of  floor(A[i][kb] * 2^32) * num_c(i, kb) / den(i, kb)      (integer arithmetic)
 * with den = visible keys of the block (j <= i) and num = how many of them the candidate's mask row i selects
 * (A-shape: closed form; vertical-slash: all if the block diagonal is in D, else the selected columns of the block;
 * block-sparse: all if the block is among the top-k_b pooled scores of the row's query block; dense: all).
 *   idx_eval   the evaluation-layout index set written by rs_build_indices(choice = NULL)
 *   covmix     device uint64 [n_items][n_cand][4] out: the sums per row subset (cleared by the call)
 * rows, r, sub_bounds, n_sub as for rs_probe_pooled. */
int rs_mixture_coverage(const rs_problem* p, const rs_candidate* lib, int n_cand, const float* A,
                        const int32_t* rows, int r, const int32_t* sub_bounds, int n_sub,
                        const rs_index_set* idx_eval, const float* qpool, const float* kpool,
                        uint64_t* covmix, int32_t* status, void* stream);

/* Calibrated predictor e of Eq. 4 (Section 3.3: "a small monotone regressor fitted offline from dense calibration
 * runs; it consumes only the probe descriptors and candidate metadata").  The form used here, this library's choice:
 *   z(item, c) = w0 (1 - m_hat) + w1 u + w2 entropy + w3 (1 - local) + w4 (1 - agreement) + w5 (1 - pairs / dense pairs)
 *   e(item, c) = table value of the last breakpoint z_k <= z (0 below the first; a non-decreasing step function),
 * with w >= 0 and a non-decreasing table, so e is monotone in every feature.  Dense candidates get e = 0.
 * All arithmetic is IEEE double, one rounding per operation, in the order written above.
 *   stats  device rs_cand_stats[n_items][n_cand] (rs_build_indices);  descr  device fp32 [n_items][4] (rs_probe_pooled)
 *   w      HOST double[6];  bp_z, bp_e  HOST double[n_bp] (n_bp <= 64, bp_z ascending)
 *   e_out  device double[n_items][n_cand] */
int rs_regressor_eval(const rs_problem* p, const rs_candidate* lib, int n_cand, const rs_cand_stats* stats,
                      const float* descr, const double* w, const double* bp_z, const double* bp_e, int n_bp,
                      double* e_out, int32_t* status, void* stream);

/* Offline calibration of Section 3.5 and the predictor e of Section 3.3 / Eq. 4 from audit records (HOST function, host
 * arrays; a few hundred records, run once per model / library / length bucket):
 *   features [n_records][n_features], target [n_records] (audited error, e.g. mean row error / V_max),
 *   residual [n_records] (m_hat - m_true of the audited (head, candidate)), q in (0, 1]
 * Outputs: delta_q = the ceil(q n)-th smallest residual floored at 0 ("a one-sided residual quantile", Section 3.3);
 *   w [n_features] >= 0 minimising ||features w - target||^2 (w = e_0 when the minimiser is 0); the non-decreasing
 *   least-squares step function of target on z = features . w as breakpoints bp_z (ascending) / bp_e (non-decreasing),
 *   thinned to at most max_breakpoints (<= 64 for rs_regressor_eval) by dropping the smallest jumps; n_bp their number.
 *   bp_z, bp_e need room for n_records entries. */
int rs_calibration_fit(int n_records, int n_features, const double* features, const double* target,
                       const double* residual, double q, int max_breakpoints, double* delta_q, double* w,
                       double* bp_z, double* bp_e, int* n_bp);

/* Measured latency table of Section 3.1 ("we profile every (p, b, n) tuple"): cand_ms [n_cand] = measured time of one
 * attention launch with every item routed to candidate c; it is split over the items in proportion to their exact
 * pair counts pairs [n_items][n_cand] and written as integer nanoseconds (>= 1) to table [n_items][n_cand], the
 * `cost` argument of rs_route.  HOST function, host arrays. */
int rs_cost_table_from_times(int n_items, int n_cand, const double* cand_ms, const uint64_t* pairs, int64_t* table);

/* Dense audit of Section 3.5: row-wise output error between two attention outputs of the same shape,
 *   err[i] = || Oa_i - Ob_i ||_2,  norm_a[i] = || Oa_i ||_2   (fp32 accumulation over the 128 dimensions)
 * Oa, Ob: [n_rows][128] bf16 (o_dtype 0) or fp32 (o_dtype 1); err, norm_a (may be NULL): device fp32[n_rows]. */
int rs_output_error(long long n_rows, const void* Oa, const void* Ob, int o_dtype, float* err, float* norm_a,
                    int32_t* status, void* stream);

/* The whole hot path of one layer in one call (the procedure table of Section 3.4): rs_probe (pooling all of Q
 * deferred), rs_build_indices in evaluation mode, rs_route, rs_pool_queries, rs_build_indices for the routed
 * block-sparse rows, one rs_sparse_prefill_attn launch, rs_certificate on the probe rows.  Host code only: it
 * enqueues those calls on `stream` in that order with the arguments below; the routes never leave the device, so the
 * call returns before any kernel has run and can be captured into a CUDA graph.  Results are the same, bit for bit,
 * as issuing the seven calls one by one.
 *   params      as for rs_route.  params->fixed_choice != NULL skips candidate evaluation (stats are not written) and
 *               runs the given routes; otherwise routing is online and idx_eval must be in the evaluation layout
 *   cost        as for rs_route (NULL: 512 x selected pairs)
 *   b           device buffers, all owned by the caller; shapes as documented at the call that fills them.
 *               descr, report, onorm, counters, probe_rows (with m_row, cert_row, m_head, cert_head) may be NULL;
 *               without probe_rows or onorm the certificate step is skipped.  probe_rows: the last 64 rows of every
 *               segment, segment after segment (the layout of lse_probe); vmax of the last segment bounds Eq. 5
 *   ws          one workspace of rs_workspace_bytes() bytes serves every step
 * Errors: the first failing step's code; kernels of earlier steps stay enqueued. */
typedef struct {
  float *vert, *slash, *lse_probe, *qpool, *kpool, *vmax, *descr;
  rs_cand_stats* stats;
  rs_index_set idx_eval;       /* evaluation layout (n_vs_slots = n_items * n_cand) */
  rs_index_set idx;            /* materialised layout */
  int32_t* choice;             /* [n_items] out */
  rs_route_report* report;
  void* O; int32_t o_dtype;    /* 0: bf16, 1: fp32 */
  int32_t n_probe_rows;
  float *lse_sel, *onorm;
  uint64_t* counters;
  const int32_t* probe_rows;
  float *m_row, *cert_row, *m_head, *cert_head;
} rs_layer_buffers;
int rs_routed_prefill_layer(const rs_problem* p, const void* Q, const void* K, const void* V,
                            const rs_candidate* lib, int n_cand, const rs_route_params* params,
                            const int64_t* cost, const rs_layer_buffers* b, void* ws, size_t ws_bytes,
                            int32_t* status, void* stream);

/* The producer of Q, K, V with the probe's streaming reductions fused into it (Section 3.4: the routing work "runs on
 * the CPU concurrently with projection kernels or as a fused GPU reduction").  One layer's QKV projection
 *   Y = X W^T,   X [n_tokens][d_model] bf16,   W [(n_q_heads + 2 n_kv_heads) * 128][d_model] bf16, rows ordered
 *   Q head 0.., K head 0.., V head 0..  (each head 128 consecutive rows)
 * on the tensor cores, the rotary embedding of Q and K in the "rotate half" pairing (dimension i with i + 64):
 *   out[i] = y[i] cos[t][i] - y[i + 64] sin[t][i],  out[i + 64] = y[i + 64] cos[t][i] + y[i] sin[t][i],
 * rope_cos / rope_sin device fp32 [n_tokens][64]; V is not rotated.  Q, K, V are written as bf16 [heads][n_tokens][128]
 * (the layout every other call takes), rounded once to nearest even from the fp32 accumulator.
 * Side outputs (each may be NULL), formed from the ROUNDED values so that they equal what rs_probe would compute
 * from the tensors just written (up to the order of fp32 additions):
 *   qpool [n_q_heads][n_tokens/64][128], kpool [n_kv_heads][n_tokens/64][128]   64-row means (Section 3.1: "pooled
 *         queries and keys score coarse blocks")
 *   vbmax [n_kv_heads][n_tokens/64]   max over the block's rows of ||v||_2^2 (Eq. 5 needs V_max = max_j ||v_j||;
 *         rs_value_norm_max turns it into rs_probe's vmax)
 * A caller that has them passes NULL for qpool, kpool and vmax to rs_probe, which then skips its own pooling of K and
 * its pass over V.  n_tokens a multiple of 64, d_model a multiple of 64, n_q_heads and n_kv_heads even.
 * Errors as for the other calls; nothing is allocated; the kernel's waits are bounded (RS_ERR_TIMEOUT in status). */
int rs_qkv_rope_project(int n_tokens, int d_model, int n_q_heads, int n_kv_heads, const void* X, const void* W,
                        const float* rope_cos, const float* rope_sin, void* Q, void* K, void* V,
                        float* qpool, float* kpool, float* vbmax, int32_t* status, void* stream);

/* vmax [n_seg][n_kv_heads] of rs_probe (V_max of Eq. 5 per segment: sqrt of the largest ||v_j||^2 over the keys below
 * the segment's end) from the block maxima vbmax [n_kv_heads][n_keys/64] written by rs_qkv_rope_project. */
int rs_value_norm_max(const rs_problem* p, const float* vbmax, float* vmax, int32_t* status, void* stream);

/* Self test of the bounded device-side wait every kernel of this library uses (no passage of the paper: the waits
 * exist because the kernels synchronise TMA, tensor-core and softmax roles through mbarriers).  Launches one small
 * kernel that waits on a barrier nothing arrives on, with a limit of poll_limit (1 .. 2^20) polls; the wait gives up,
 * the kernel writes RS_ERR_TIMEOUT and site 99 to `status` (device int32[RS_STATUS_WORDS], required) and ends
 * normally, leaving the context usable. */
int rs_selftest_wait_timeout(int32_t* status, unsigned int poll_limit, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ROUTESPARSE_H_ */
