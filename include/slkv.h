/*
 * slkv.h -- C ABI of the SurfaceLogicKV prefill KV-cache compression library (CUDA, sm_100a).
 *
 * One call per step of the paper's method:
 *   slkv_behavior_scores Stage 1, SF_sc / LG_sc / INF_sc of attention rows               (Sec. 3.2, Algorithm 1)
 *   slkv_alloc_budgets   Stage 2, per-head KV budgets from the INF_sc table     (Sec. 3.3, Eq. 6, Algorithm 2)
 *   slkv_score           relevance of every history key to the query window     (Sec. 3.4, Eq. 7, Alg. 3 l.4-6)
 *   slkv_compress        score -> top-(C - window) history rows + window, gather (Sec. 3.4, Eq. 8, Algorithm 3)
 *   slkv_compress_host   the same, from/to host buffers (copies included)
 *   slkv_compress_overlapped / slkv_join   the same, successive layers overlapped on the GPU
 *   slkv_cp_*            the same for one sequence whose keys are split over ranks (context parallel)
 *   slkv_row_lse         the window rows' log-sum-exp over their softmax domain       (Eq. 3-4, Eq. 7)
 *
 * Conventions
 *   - "dev" pointers are device memory of the current CUDA device, "host" pointers are host memory.
 *   - The caller owns every buffer.  The library allocates no device memory; scratch comes from the
 *     caller's `workspace` (size from slkv_workspace_bytes) and must stay untouched until the enqueued
 *     work has finished.  Nothing is freed or retained by the library.  One exception, for callers that
 *     have no workspace to give: slkv_score_noalloc works in a fixed array of SLKV_NOALLOC_SCRATCH_BYTES
 *     that is part of the library's device image (see there for when it comes into being and how long it
 *     lives).
 *   - All device work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *     No call synchronises the device except slkv_compress_host, which returns after its results are
 *     in the host buffers.
 *   - Every function returns SLKV_OK (0) or a negative slkv_status.  Argument errors are found on the
 *     host before anything is enqueued.  Errors only visible in device data (a negative INF_sc, an
 *     output capacity that turns out too small) are written to the optional device word `status`
 *     (untouched when nothing is wrong -- zero it first), never raised as a device fault.
 *
 * Tensor layouts (element = float for SLKV_F32, bfloat16 for SLKV_BF16; head_dim contiguous)
 *   K, V   packed varlen, token-major: element (t, h, p) at t*stride_tok + h*stride_head + p,
 *          t in [0, total_tokens), sequences delimited by cu_seqlens[n_seqs+1] (cu[0] = 0).
 *   Q_win  the queries of each sequence's last `window` tokens: element (s, i, h, p) at
 *          s*q_stride_seq + i*q_stride_row + h*q_stride_head + p; row i is token len_s - window + i.
 *          (Rows are unused for sequences not longer than the window.)
 *   GQA    query head h scores against KV head h / (n_q_heads / n_kv_heads).
 *   pooled ragged float array: sequence s, KV head h, history position j (j < n_hist_s = max(len_s -
 *          window, 0)) at  n_kv_heads * sum_{s'<s} n_hist_s'  +  h * n_hist_s  +  j.
 *   packed output: segment seg = s*n_kv_heads + h owns rows offsets[seg] .. offsets[seg+1]-1 of k_out /
 *          v_out / kept_idx; its rows are the selected history positions in ascending order followed by
 *          the window positions; a row is head_dim contiguous elements.  kept_idx holds positions
 *          within the sequence (0-based).
 */
#ifndef SLKV_H_
#define SLKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum slkv_status {
  SLKV_OK = 0,
  SLKV_ERR_NULL_PTR = -1,       /* a required pointer is NULL */
  SLKV_ERR_BAD_SHAPE = -2,      /* a size / count / stride is out of the supported range */
  SLKV_ERR_BAD_DTYPE = -3,      /* dtype / mode enum not recognised or not supported by the chosen path */
  SLKV_ERR_BAD_ALIGN = -4,      /* a pointer or stride breaks the 16-byte row alignment rule */
  SLKV_ERR_BUDGET_SUM = -5,     /* total < n_layers*n_heads*fixed, or fixed < 0 */
  SLKV_ERR_NEG_INF_SC = -6,     /* an INF_sc entry is negative or not finite (device status word) */
  SLKV_ERR_CAPACITY = -7,       /* out_capacity_rows smaller than the rows to write */
  SLKV_ERR_WORKSPACE = -8,      /* workspace NULL or smaller than slkv_workspace_bytes */
  SLKV_ERR_CUDA = -9,           /* a CUDA runtime call failed (see slkv_last_cuda_error) */
  SLKV_ERR_DEVICE_TIMEOUT = -10 /* a bounded device-side wait ran out (device status word) */
} slkv_status;

enum { SLKV_F32 = 0, SLKV_BF16 = 1 };                 /* slkv_params.dtype */
enum { SLKV_POOL_MAX = 0, SLKV_POOL_AVG = 1 };        /* slkv_params.pool_mode */
enum { SLKV_HISTORY = 0,                              /* slkv_params.softmax_domain: softmax over the history keys */
       SLKV_ALL_CAUSAL = 1 };                         /*   over every key a window query sees causally */
enum { SLKV_LSE_LN = 0, SLKV_LSE_LOG2 = 1 };          /* slkv_params.lse_units: natural log / base-2 log */
enum { SLKV_PATH_AUTO = 0,                            /* slkv_params.score_path */
       SLKV_PATH_SIMT = 1,                            /*   fp32 FMA kernels (any dtype, head_dim 64/128) */
       SLKV_PATH_TENSOR = 2 };                        /*   tcgen05 + TMA kernels (bf16, head_dim 128) */

/* Shapes and options shared by slkv_score / slkv_compress. Strides are in elements. */
typedef struct slkv_params {
  int32_t n_seqs;          /* >= 1 */
  int32_t n_q_heads;       /* multiple of n_kv_heads */
  int32_t n_kv_heads;
  int32_t head_dim;        /* 64 or 128 */
  int32_t window;          /* w >= 1: observation window (last w tokens), always kept */
  int32_t pool_kernel;     /* odd >= 1 (1 = no pooling) */
  int32_t dtype;           /* SLKV_F32 | SLKV_BF16: element type of Q_win, K, V and the packed outputs */
  int32_t pool_mode;       /* SLKV_POOL_MAX | SLKV_POOL_AVG */
  int32_t softmax_domain;  /* SLKV_HISTORY | SLKV_ALL_CAUSAL: the keys a window row's softmax runs over */
  int32_t score_path;      /* SLKV_PATH_AUTO picks TENSOR when the shape allows it, else SIMT */
  int32_t lse_units;       /* SLKV_LSE_LN | SLKV_LSE_LOG2: units of lse_opt / slkv_row_lse's output */
  int32_t history_only;    /* 0: the last `window` rows of every sequence in K / V are the window rows (never scored);
                              1: K holds history rows only -- a range of a longer sequence's keys whose window rows
                              live elsewhere (context-parallel sharding).  n_seqs must be 1; taken by slkv_score,
                              slkv_row_lse and slkv_score_noalloc, SLKV_ERR_BAD_SHAPE from the compress entry points;
                              the softmax then runs over the rows given, whatever softmax_domain says */
  int64_t k_stride_tok, k_stride_head;
  int64_t v_stride_tok, v_stride_head;
  int64_t q_stride_seq, q_stride_row, q_stride_head;
} slkv_params;

/* Human-readable name of a status code (static string, never NULL). */
const char* slkv_strerror(int status);

/* Last CUDA runtime error code seen by a call that returned SLKV_ERR_CUDA on this thread (0 = none). */
int slkv_last_cuda_error(void);

/*
 * Stage-1 attention behaviour analysis (Sec. 3.2, Algorithm 1), for a batch of attention rows (one row = the
 * attention weights of one head for one probe prompt's answering position, over the context).
 * For each row with needle positions N and top-k positions T (both as sets):
 *     WO = sum of W over N and T,  WD = sum over T without N,  TNW = sum over N,  WS = max(0, TNW - WO)
 *     SF_sc = WO / (WO + WD),  LG_sc = WO / (WO + WS),  INF_sc = 2 SF_sc LG_sc / (SF_sc + LG_sc)     (0/0 = 0)
 *   attn         dev, float: row r starts at attn + r*row_stride and has row_len weights (row_stride 0 shares one row)
 *   needle_idx   dev, int32: row r's needle positions at needle_idx + r*needle_stride, n_needle entries
 *                (needle_stride 0: one list for all rows); entries outside [0, row_len) are padding
 *   topk_idx     dev, int32: likewise the positions of the row's k largest weights (n_topk entries, topk_stride)
 *   sf_sc, lg_sc, inf_sc   dev, out, float[n_rows]
 * An index listed twice counts once.  Averaging the per-row scores into the per-(layer, head) INF_sc table that
 * slkv_alloc_budgets takes is left to the caller (the paper does not print how it aggregates over prompts).
 * Limits: n_needle, n_topk <= 4096.
 */
int slkv_behavior_scores(const float* attn, int64_t n_rows, int32_t row_len, int64_t row_stride,
                         const int32_t* needle_idx, int32_t n_needle, int64_t needle_stride, const int32_t* topk_idx,
                         int32_t n_topk, int64_t topk_stride, float* sf_sc, float* lg_sc, float* inf_sc, void* stream);

/*
 * Stage-2 budget allocation (Sec. 3.3, Eq. 6; Algorithm 2).
 *   inf_sc   dev, float[n_layers*n_heads], row-major (layer, head); INF_sc >= 0, finite
 *   fixed    fixed part every head receives (= b_c (1 - 1/beta) in the paper's notation)
 *   total    sum of all budgets (= b_c * n_layers * n_heads); dynamic pool D = total - N*fixed >= 0
 *   budgets  dev, out, int32[n_layers*n_heads]
 *   status   dev, optional: set to SLKV_ERR_NEG_INF_SC (budgets then left unwritten)
 * Head (i, j) receives fixed + its share of D in proportion to Algorithm 2's weight
 * (0.01 + L_i/L_s) * (inf_ij/L_s), L_i the layer's INF_sc sum, L_s the grand sum; shares are rounded by
 * largest remainder (ties: lower index first) so that the budgets sum to `total` exactly.  All-zero
 * INF_sc gives uniform shares.  fp64 arithmetic in a fixed order: results are reproducible bit for bit.
 * Limits: n_layers <= 1024, n_layers*n_heads <= 16384, total < 2^31 (else SLKV_ERR_BAD_SHAPE).
 */
int slkv_alloc_budgets(const float* inf_sc, int32_t n_layers, int32_t n_heads, int32_t fixed, int64_t total,
                       int32_t* budgets, int32_t* status, void* stream);

/*
 * The same allocation with the readings Sec. 3.3 leaves open (Eq. 6 and its prose; Algorithm 2's last line).
 *   head_normaliser  SLKV_NORM_GLOBAL: a head's share S_ij = inf_ij / L_s of the grand sum, as Algorithm 2 prints it;
 *                    SLKV_NORM_WITHIN_LAYER: inf_ij / L_i of its own layer's sum, as the prose under Eq. 6 describes
 *                    it (an all-zero layer shares evenly).  Under the second one a layer's total follows
 *                    (0.01 + L_i/L_s) / (1 + 0.01 n_layers): the 0.01 "minimum layer budget" really is a floor.
 *   rounding         SLKV_ROUND_SUM_EXACT: normalised weights, largest remainder, sum == total (as slkv_alloc_budgets);
 *                    SLKV_ROUND_PAPER: Algorithm 2's own C = floor(max(0, fixed + D * weight) + 0.5) per head with
 *                    D = total - N*fixed; the weights are not normalised, so the sum is whatever it comes to.
 *   cap              0: none.  > 0: no head gets more than `cap` (say, the sequence length: budget beyond it could
 *                    never be used).  With SLKV_ROUND_SUM_EXACT what a full head cannot take goes to the others in
 *                    proportion to their weights, again and again until nobody is above the cap, and the budgets
 *                    still sum to `total` (needs cap >= fixed and total <= N * cap, else SLKV_ERR_BUDGET_SUM); with
 *                    SLKV_ROUND_PAPER the budgets are just clipped.  The paper has no cap.
 * opt == NULL means {SLKV_NORM_GLOBAL, SLKV_ROUND_SUM_EXACT, 0}.  Other arguments, limits and errors as
 * slkv_alloc_budgets; an unknown enum value gives SLKV_ERR_BAD_DTYPE.  Bit-reproducible like slkv_alloc_budgets.
 */
enum { SLKV_NORM_GLOBAL = 0, SLKV_NORM_WITHIN_LAYER = 1 };     /* slkv_alloc_options.head_normaliser */
enum { SLKV_ROUND_SUM_EXACT = 0, SLKV_ROUND_PAPER = 1 };       /* slkv_alloc_options.rounding */
typedef struct slkv_alloc_options {
  int32_t head_normaliser;
  int32_t rounding;
  int64_t cap;
} slkv_alloc_options;
int slkv_alloc_budgets_ex(const float* inf_sc, int32_t n_layers, int32_t n_heads, int32_t fixed, int64_t total,
                          const slkv_alloc_options* opt, int32_t* budgets, int32_t* status, void* stream);

/* Bytes of workspace slkv_score / slkv_compress need for these shapes (0 on invalid arguments).
 * cu_seqlens_host: host, int32[n_seqs+1]. */
size_t slkv_workspace_bytes(const slkv_params* p, const int32_t* cu_seqlens_host);

/* Number of floats in the ragged `pooled` array: n_kv_heads * sum_s max(len_s - window, 0) (-1 on error). */
int64_t slkv_pooled_elems(const slkv_params* p, const int32_t* cu_seqlens_host);

/* Upper bound of packed rows for any budgets: n_kv_heads * total_tokens (-1 on error). */
int64_t slkv_packed_rows_upper_bound(const slkv_params* p, const int32_t* cu_seqlens_host);

/*
 * Relevance scores (Sec. 3.4, Eq. 7; Algorithm 3 lines 4-6; scale and softmax axis from Eq. 3-4).
 * For every sequence s, KV head g and history key j < n_hist_s:
 *     vote[j]   = (1/G) * sum_{query heads h of group g} sum_{window rows i} exp(q_i . k_j / sqrt(head_dim) - lse_i)
 *     pooled[j] = max (or zero-padded mean) of vote over [j - pool_kernel/2, j + pool_kernel/2] within the history
 * where lse_i is the log-sum-exp of row i's scaled scores over its softmax domain: the history keys
 * (SLKV_HISTORY: Eq. 7 and Algorithm 3 as printed) or the history keys plus the window keys up to the
 * row's own position (SLKV_ALL_CAUSAL: the prefill attention's own softmax, the reading of the prior work
 * Sec. 3.4 refers to; the window columns get no vote).  (The paper leaves the reduction over the window
 * rows, the GQA reduction and the pooling to prior work; this is the reading used here.)
 *   q_win, k         dev, layouts above
 *   cu_seqlens_dev   dev, int32[n_seqs+1];  cu_seqlens_host: the same values on the host (sizes the launch)
 *   lse_opt          dev, optional, float[n_seqs][n_q_heads][window] in p->lse_units: the rows' log-sum-exp
 *                    when the caller has it already (a prefill attention kernel that keeps its softmax
 *                    statistics has exactly the SLKV_ALL_CAUSAL one).  NULL: computed here, which costs a
 *                    second pass over K.  The values are used as given, whatever softmax_domain says.
 *   pooled           dev, out, float[slkv_pooled_elems]
 *   status           dev, optional: SLKV_ERR_DEVICE_TIMEOUT if a bounded wait inside a kernel ran out
 *                    (pooled is then incomplete)
 * Accuracy: fp32 accumulation; relative error of pooled <= 1e-3 of the exact value.
 */
int slkv_score(const slkv_params* p, const void* q_win, const void* k, const int32_t* cu_seqlens_dev,
               const int32_t* cu_seqlens_host, const float* lse_opt, float* pooled, int32_t* status,
               void* workspace, size_t workspace_bytes, void* stream);

/*
 * The row statistics alone (Eq. 3-4 with Eq. 7's key set): lse_out[s][h][i] = log sum_j exp(q_i . k_j /
 * sqrt(head_dim)) over the softmax domain of p->softmax_domain, in p->lse_units, for the window rows of
 * every sequence longer than the window (rows of shorter sequences are left untouched).  It is what
 * slkv_score computes first when lse_opt is NULL; fed back as lse_opt it reproduces that call bit for bit
 * with SLKV_LSE_LOG2 (the kernels' own unit), and to rounding with SLKV_LSE_LN.  Callers that shard the
 * keys of one sequence over several devices merge these per shard and pass the result as lse_opt.
 *   lse_out   dev, out, float[n_seqs][n_q_heads][window]
 * Other arguments and errors as slkv_score.
 */
int slkv_row_lse(const slkv_params* p, const void* q_win, const void* k, const int32_t* cu_seqlens_dev,
                 const int32_t* cu_seqlens_host, float* lse_out, int32_t* status, void* workspace,
                 size_t workspace_bytes, void* stream);

/*
 * KV entry selection and gather for one layer (Sec. 3.4, Eq. 8; Algorithm 3).
 * For each segment (s, h) with budget C = budgets[h]:  kept = min(len_s, max(C, window)) rows survive:
 * everything if len_s <= C (Alg. 3 l.1-3), else the window rows plus the kept - window history positions
 * with the largest pooled score (ties: lower position first), in ascending position order (l.7-10).
 *   budgets            dev, int32[n_kv_heads]: this layer's row of slkv_alloc_budgets' output
 *   lse_opt            dev, optional: as in slkv_score
 *   k_out, v_out       dev, out, [out_capacity_rows, head_dim] elements of p->dtype
 *   offsets            dev, out, int32[n_seqs*n_kv_heads + 1]
 *   kept_idx           dev, out, int32[out_capacity_rows]
 *   pooled_opt         dev, optional out, float[slkv_pooled_elems]: the scores the selection used
 *   status             dev, optional: SLKV_ERR_CAPACITY if offsets[last] > out_capacity_rows (rows beyond
 *                      the capacity are then not written; offsets are still complete)
 * Gathered rows are bit copies of the input rows.
 */
int slkv_compress(const slkv_params* p, const void* q_win, const void* k, const void* v,
                  const int32_t* cu_seqlens_dev, const int32_t* cu_seqlens_host, const int32_t* budgets,
                  const float* lse_opt, void* k_out, void* v_out, int64_t out_capacity_rows, int32_t* offsets, int32_t* kept_idx,
                  float* pooled_opt, int32_t* status, void* workspace, size_t workspace_bytes, void* stream);

/*
 * slkv_compress with the calls of successive layers overlapped on the GPU (Algorithm 3, same results).
 *
 * The layers of a prefill are independent problems, and inside one layer the vote pass needs every key's row
 * statistics first (the softmax of Eq. 7 runs over all keys).  This entry point therefore works on several layers
 * at once: the score kernel takes a LIST of layers per launch and runs, in every CTA, the row-statistics pass of a
 * layer beside the vote pass of the layer before it; the selection and the gather of a layer run on side streams
 * of the library's own while the score kernel works on later layers.  A call queues its layer; the score kernel
 * goes out when eight layers are queued and a ninth arrives, or at slkv_join.  Consequences:
 *   - Nothing of a call needs to have been enqueued when it returns, and its outputs (k_out, v_out, offsets,
 *     kept_idx, pooled_opt, status) are NOT ordered on `stream`.  slkv_join(stream) enqueues whatever is still
 *     queued and makes `stream` wait for every overlapped call made so far on the current device (no host wait);
 *     consume outputs, or free / overwrite any input, output or workspace buffer -- q_win, k, v, cu_seqlens_dev
 *     and budgets included -- only behind it.  cu_seqlens_host is read during the call only.  Any other slkv_*
 *     call that uses a workspace joins by itself first.
 *   - Streams and host threads: the calls made on one stream form one sequence (queue, workspace slots, events);
 *     calls made on another stream -- by another host thread or the same one -- form another, and the two do not
 *     disturb each other as long as each has its own workspace (calls on two streams that share a workspace are
 *     serialised: the later one waits for what the other stream has in flight).  A join orders its stream behind
 *     the calls of every stream but settles only its own stream's: each stream that consumes results joins for
 *     itself.  The entry points may be called from several host threads at once (one lock inside); up to eight
 *     streams per device keep a sequence each, a ninth takes over the one used longest ago once that one's
 *     stream has been made to wait for what it had in flight.
 *   - workspace must hold slkv_workspace_bytes_overlapped: votes, source-row lists and row statistics for up to
 *     eighteen layers in flight (77 MB for 8 KV heads x 32k keys; three layers' worth for shapes the list kernel
 *     does not take).  Successive calls share one workspace; a call with another shape or workspace first drains
 *     what is in flight.  q_win, k, v, budgets and the outputs of calls that may be in flight together must not
 *     alias each other's outputs.
 *   - The first call on a stream creates eighteen side streams and 54 events for it (no device memory).
 *   - The call sequence is stream-ordered and allocates nothing, so a step's calls plus the join can be captured
 *     in a CUDA graph (the side streams fork from and rejoin `stream`).
 *   - The list kernel takes bf16, head_dim 128, (n_q_heads / n_kv_heads) * window <= 128 and a multiple of 32,
 *     at most 64 sequences, segments of at most 32768 history positions, pool_kernel <= 9.  Other shapes that the
 *     one-CTA selection takes run one layer per score launch with the selection and gather on the side streams;
 *     the rest run as slkv_compress does, on `stream`, after a join.
 * Arguments, results and error codes otherwise as slkv_compress.
 */
int slkv_compress_overlapped(const slkv_params* p, const void* q_win, const void* k, const void* v,
                             const int32_t* cu_seqlens_dev, const int32_t* cu_seqlens_host, const int32_t* budgets,
                             const float* lse_opt, void* k_out, void* v_out, int64_t out_capacity_rows, int32_t* offsets,
                             int32_t* kept_idx, float* pooled_opt, int32_t* status, void* workspace,
                             size_t workspace_bytes, void* stream);
size_t slkv_workspace_bytes_overlapped(const slkv_params* p, const int32_t* cu_seqlens_host);
/* Enqueues the layers still queued by slkv_compress_overlapped and orders `stream` after every overlapped call made
 * so far on the current device (see above). */
int slkv_join(void* stream);

/*
 * Context-parallel compression of ONE long sequence whose history keys are split over ranks (Sec. 3.4, Eq. 7-8;
 * Algorithm 3; same kept set as slkv_compress on the whole sequence, up to the score tolerance).
 *
 * Rank r of n_parts holds K / V rows of a contiguous range of history positions [b_r, e_r) plus up to pool_kernel/2
 * rows of each neighbour's range on either side (so that pooling needs nothing from the neighbours); the last rank
 * also holds the `window` rows behind the history.  Every rank holds q_win.  Per layer, on every rank:
 *   1. slkv_row_lse over the rows it OWNS (history_only = 1 on all ranks but the last, whose range is an ordinary
 *      sequence tail): the rows' log-sum-exp over this rank's keys.            all-gather over ranks
 *   2. slkv_cp_merge_lse: log-sum-exp over the ranks = the rows' log-sum-exp over all keys.
 *   3. slkv_score with lse_opt = that, over the owned rows plus the neighbours' margins: pooled scores.
 *   4. slkv_cp_select_init once, then for level = 0, 1, 2: slkv_cp_histogram over the owned positions,
 *      all-reduce (sum) of the histograms over ranks, slkv_cp_descend on the sum.  prefix[] then holds the bit
 *      pattern of every head's threshold score, need[] how many positions with exactly that score are kept.
 *   5. slkv_cp_local_ties (from the rank's OWN level-2 histogram): all-gather over ranks; slkv_cp_emit packs the
 *      rank's kept rows (the ties go to the lowest positions, i.e. in rank order) and its window rows.
 * The packed cache of head h is the concatenation over ranks of each rank's rows of head h; offsets[] are local.
 * The collectives (two all-gathers of a few hundred bytes and three all-reduces of n_kv_heads x 2048 int32 per layer)
 * are the caller's: the library launches no communication.  Everything is enqueued on `stream`; all pointers are
 * device pointers unless stated.
 *   lse_parts  [n_parts][n_q_heads][window] in p->lse_units (-inf for a rank without keys); lse_out [n_q_heads][window]
 *   prefix, need, ties  [n_kv_heads]; hist  [n_kv_heads][2048] int32 (zeroed by slkv_cp_histogram)
 *   pooled     [n_kv_heads][row_stride]: slkv_score's output for this rank's rows; the owned positions are
 *              own_begin .. own_begin + own_count - 1 of every row (the margins before and after them are not owned)
 *   pos0       position in the whole sequence of the first owned row
 *   rows       rows of k / v on this rank; row j of k / v is position j of pooled; window_rows = 0, or on the last rank
 *              the number of window rows, which are the last window_rows rows of k / v at positions window_pos0 ..
 *   ties_all   [n_parts][n_kv_heads]: every rank's slkv_cp_local_ties; part = this rank's index
 *   offsets    out, int32[n_kv_heads + 1]; kept_idx out, positions in the whole sequence; k_out, v_out as slkv_compress
 *   status     optional: SLKV_ERR_CAPACITY if offsets[n_kv_heads] > out_capacity_rows
 */
int slkv_cp_merge_lse(const slkv_params* p, const float* lse_parts, int32_t n_parts, float* lse_out, void* stream);
int slkv_cp_select_init(const int32_t* budgets, int32_t n_kv_heads, int32_t window, int64_t seq_len, uint32_t* prefix,
                        int32_t* need, void* stream);
int slkv_cp_histogram(const float* pooled, int32_t n_kv_heads, int64_t row_stride, int32_t own_begin, int32_t own_count,
                      int32_t level, const uint32_t* prefix, int32_t* hist, void* stream);
int slkv_cp_descend(const int32_t* hist, int32_t n_kv_heads, int32_t level, uint32_t* prefix, int32_t* need,
                    void* stream);
int slkv_cp_local_ties(const int32_t* hist_local, const uint32_t* prefix, int32_t n_kv_heads, int32_t* ties,
                       void* stream);
size_t slkv_cp_workspace_bytes(int32_t n_kv_heads, int32_t own_count, int64_t out_capacity_rows);
int slkv_cp_emit(const slkv_params* p, const void* k, const void* v, int64_t rows, const float* pooled,
                 int64_t row_stride, int32_t own_begin, int32_t own_count, int64_t pos0, const uint32_t* threshold,
                 const int32_t* need, const int32_t* ties_all, int32_t n_parts, int32_t part, int32_t window_rows,
                 int64_t window_pos0, void* k_out, void* v_out, int64_t out_capacity_rows, int32_t* offsets,
                 int32_t* kept_idx, int32_t* status, void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of device arena slkv_compress_host needs (inputs, outputs and workspace; 0 on invalid arguments). */
size_t slkv_compress_host_arena_bytes(const slkv_params* p, const int32_t* cu_seqlens_host,
                                      int64_t out_capacity_rows);

/*
 * slkv_compress for callers whose tensors live in host memory (Algorithm 3, same semantics).
 * q_win, k, v, budgets are HOST inputs (dense layouts: the strides in `p` must describe contiguous
 * [n_seqs, window, n_q_heads, head_dim] and [total_tokens, n_kv_heads, head_dim] arrays); k_out, v_out,
 * offsets, kept_idx are HOST outputs.  `arena` is caller-owned DEVICE memory of at least
 * slkv_compress_host_arena_bytes, 256-byte aligned.  The call copies the inputs to the arena, runs the
 * kernels, copies offsets, kept_idx and the packed rows back and waits for `stream` before returning, so
 * the outputs are valid on return.  Pinned host buffers make the copies asynchronous and fast; pageable
 * ones work.  Returns SLKV_ERR_CAPACITY if out_capacity_rows is too small (nothing is copied back then
 * except offsets).  *rows_out (optional) receives offsets[last].
 */
int slkv_compress_host(const slkv_params* p, const void* q_win, const void* k, const void* v,
                       const int32_t* cu_seqlens_host, const int32_t* budgets, void* k_out, void* v_out,
                       int64_t out_capacity_rows, int32_t* offsets, int32_t* kept_idx, int64_t* rows_out,
                       void* arena, size_t arena_bytes, void* stream);

/*
 * slkv_score without a workspace argument, for callers that cannot allocate device memory.  (The paper has
 * no counterpart: this is a property of the library, not of the method.)
 *
 * Who needs it: code that runs inside a host application which has already handed every free byte of the
 * GPU to its own pool (a serving engine that sizes its KV-cache blocks from "all memory that is left"), or a
 * plug-in that is given tensors but no handle to the host's allocator.  There cudaMalloc fails, or succeeds
 * only by synchronising the whole device and shrinking somebody else's pool, and torch's allocator is not
 * the caller's to use.  Such a caller still owns its inputs and outputs; what it lacks is scratch.
 *
 * The scratch is a fixed array of SLKV_NOALLOC_SCRATCH_BYTES inside the library's device image: every GPU
 * that loads the library holds that much memory until the process exits, used or not.  The call computes
 * exactly what slkv_score computes, with the same kernels and the same results.
 *   - Shapes whose slkv_workspace_bytes exceed the array are rejected with SLKV_ERR_WORKSPACE before anything
 *     is enqueued (32k tokens x 8 KV heads x 128 score rows needs about 5.3 MB).
 *   - The first call on each device looks up the array's device address (a CUDA runtime query, made with that
 *     device current) and keeps it.  With the CUDA runtime's lazy module loading the array comes into being at
 *     that query, not when the library is loaded: make the first call at start-up, while SLKV_NOALLOC_SCRATCH_BYTES
 *     of device memory are still free (otherwise it returns SLKV_ERR_CUDA), and outside any stream capture.
 *   - The library itself calls no cudaMalloc, cudaFree or other allocating routine, on the first call or later.
 *   - All calls on a device share the one array.  It keeps whatever the previous call left; nothing in it has
 *     to be zero, each call overwrites what it reads.  Two calls whose kernels may overlap on the GPU
 *     (different streams, no ordering between them) race on it: order them.
 * Arguments and return value as slkv_score, minus workspace / workspace_bytes.  If the address query fails
 * the call returns SLKV_ERR_CUDA and slkv_noalloc_last_cuda_error() gives the runtime's code.
 */
#define SLKV_NOALLOC_SCRATCH_BYTES (8u << 20)
int slkv_score_noalloc(const slkv_params* p, const void* q_win, const void* k, const int32_t* cu_seqlens_dev,
                       const int32_t* cu_seqlens_host, const float* lse_opt, float* pooled, int32_t* status,
                       void* stream);
size_t slkv_noalloc_scratch_bytes(void);      /* = SLKV_NOALLOC_SCRATCH_BYTES */
int slkv_noalloc_last_cuda_error(void);

/* Number of kernels the most recent slkv_score / slkv_compress / slkv_compress_host call on this
 * thread enqueued (launch accounting for benchmarks). */
int slkv_last_launch_count(void);

/*
 * Per-kernel timing for benchmarks (no counterpart in the paper).  While enabled on the calling thread,
 * every kernel the library enqueues is bracketed by a CUDA event pair on its stream (events are created
 * on demand and reused; this adds host work per launch, so headline timings are taken with it off).
 * on = 1: every kernel, and the overlapped entry point keeps selections and gathers on the caller's stream so that
 * the pairs do not overlap (the step is then slower than untimed); on = 2: the score kernels only, everything else
 * where it normally runs -- the score kernels' times in the regime of an untimed step; on = 0: off.
 * slkv_profile_collect waits for the recorded events, adds each kernel's elapsed milliseconds and launch
 * count into total_ms[id] / launches[id] (arrays of n_kernels entries, overwritten) and forgets the records.
 * Kernel ids run from 0 to slkv_kernel_count()-1; slkv_kernel_name gives their names.
 */
int slkv_profile_enable(int on);
int slkv_profile_collect(float* total_ms, int32_t* launches, int32_t n_kernels);
const char* slkv_kernel_name(int kernel_id);
int slkv_kernel_count(void);

/*
 * Timeline tracing of the tensor-core score kernels (diagnostics; no counterpart in the paper).
 * With a device buffer set on the calling thread, every CTA of the two score kernels stores %globaltimer
 * nanosecond stamps into it: 64 uint64 slots per CTA, pass 1 first (n_cta * 64 entries), pass 2 after
 * it.  Slots: 0 CTA start, 1 set-up done, 2 query tile landed, 3 first key tile landed, 4 CTA end,
 * 8+2i / 9+2i start / end of the softmax arithmetic on the CTA's i-th tile (i < 28).  The score kernel of the
 * overlapped entry point (a list of layers per launch, two streams per CTA) writes: 0 CTA start, 1 / 7 stream
 * A / B past its wait for the launch before, 2 first accumulator of stream A ready, 3 first log-sum-exps of
 * stream B merged, 5 / 6 stream A / B done, 4 CTA end, 8+2j / 9+2j list entry j published by stream A / begun by
 * stream B, 60 / 61 the SM cycle counter at CTA start / end.  The buffer that is set when a launch is enqueued is
 * the one it writes (the overlapped entry point enqueues a list when it is full and one more layer has come, or at
 * a join).  The buffer must hold 2 * n_cta * 64 * 8 bytes (n_cta <= number of SMs); smaller buffers switch tracing
 * off.  NULL switches it off.
 */
int slkv_trace_set_buffer(void* dev_buf, size_t bytes);

/*
 * Test hook for the bounded waits (no counterpart in the paper).  Where the CTAs of a launch wait for one another
 * (the grid-wide barrier between the two passes of slkv_score / slkv_compress, the per-layer counters of the list
 * kernel behind slkv_compress_overlapped), every wait gives up after one second, sets SLKV_ERR_DEVICE_TIMEOUT in the
 * call's status word, releases what the CTA holds and returns.  With the hook armed (on != 0) the next such launch made
 * by the calling thread waits for one arrival more than there are CTAs, so that exactly this path runs: the call's
 * results are then incomplete and its status word says so; the calls after it are unaffected.  One-shot: the launch
 * that takes it disarms it.
 */
int slkv_debug_expire_next_wait(int on);

/* Library version, major*10000 + minor*100 + patch. */
int slkv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SLKV_H_ */
