// Internal declarations shared by the translation units of libslkv (not part of the public ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "slkv.h"

namespace slkv {

constexpr double kLayerFloor = 0.01;   // minimum layer budget (Sec. 3.3)
constexpr float kLog2e = 1.4426950408889634f;

constexpr int kInlineSeqs = 64;

// Per-sequence tables: token starts (cu), exclusive prefixes of the history lengths n_hist_s and of the
// 128-key tile counts.  Batches of up to kInlineSeqs sequences carry them inside the kernel parameters
// (filled on the host from cu_seqlens_host); larger batches read the arrays a set-up kernel wrote.
struct SeqTables {
  int32_t n_inline;                       // n_seqs when the inline arrays are valid, else 0
  int32_t cu[kInlineSeqs + 1];
  int32_t tile_off[kInlineSeqs + 1];
  long long hist_off[kInlineSeqs + 1];
  const int32_t* cu_ptr;
  const int32_t* tile_ptr;
  const long long* hist_ptr;
#ifdef __CUDACC__
  __device__ __forceinline__ int cu_at(int i) const { return n_inline ? cu[i] : cu_ptr[i]; }
  __device__ __forceinline__ int tile_at(int i) const { return n_inline ? tile_off[i] : tile_ptr[i]; }
  __device__ __forceinline__ long long hist_at(int i) const { return n_inline ? hist_off[i] : hist_ptr[i]; }
#endif
};

// Where a vote pass takes the window rows' log-sum-exp from when it does not merge the row statistics of the keys
// it scored itself alone: the caller's array (lse_opt of the public entry points), and / or the statistics of the
// window keys (softmax over all causally visible keys).  Row r of a segment is query head g*G + hh, window row i with
// r = i*G + hh (head_inner) or r = hh*window + i.
struct LseSource {
  const float* lse_opt;     // [n_seqs][n_q_heads][window], or null
  const float* win_m;       // [n_seg][R] maxima (log2 units) over the window keys a row sees, or null
  const float* win_z;       // [n_seg][R] sums of 2^(x - max) over them
  float to_log2;            // lse_opt * to_log2 is in log2 units
  int n_q_heads;
#ifdef __CUDACC__
  __device__ __forceinline__ float caller_lse(int s, int g, int r, int G, int window, bool head_inner) const {
    const int hh = head_inner ? r % G : r / window;
    const int i = head_inner ? r / G : r - hh * window;
    return lse_opt[((long long)s * n_q_heads + g * G + hh) * window + i] * to_log2;
  }
#endif
};

// Programmatic dependent launch: a kernel may start while its predecessor in the stream drains; it must
// not touch global memory the predecessor may write before pdl_wait() returns.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif

// Launches `kernel` with the programmatic-serialisation attribute (and optionally a cluster shape).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              int cluster_x, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int n = 0;
  attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster_x;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Everything a score / select / gather launch needs, resolved by the host entry points.
struct Problem {
  slkv_params p;
  int G;                  // query heads per KV head
  int R;                  // score rows per KV head = G * window
  int elem;               // bytes per element
  int max_hist;           // max_s n_hist_s
  int64_t total_tokens;   // rows of K / V that exist (the extent of the K tensor map)
  int32_t cu_virtual[2];  // history_only: {0, rows + window}, the sequence the kernels are told about
  int64_t total_hist;     // sum_s n_hist_s
  int n_seg;              // n_seqs * n_kv_heads
  const int32_t* cu;      // dev
  SeqTables tab;          // per-sequence tables (inline or pointing into the workspace)
  const void* q;          // dev
  const void* k;          // dev
  const void* v;          // dev
  // workspace carve-up (dev)
  int64_t* hist_off;      // [n_seqs+1] exclusive prefix of n_hist_s
  int32_t* tile_off;      // [n_seqs+1] exclusive prefix of ceil(n_hist_s / 128)
  float* vote;            // [n_kv_heads * total_hist] ragged, same layout as pooled
  float* part_m;          // [n_seg][R][n_chunks] partial row maxima (log2 domain)
  float* part_z;          // [n_seg][R][n_chunks] partial row sums
  int n_chunks;           // chunks per segment (stride of part_*), per score path
  int chunk_keys;         // keys per chunk
  float* pooled_ws;       // [n_kv_heads * total_hist] used when the caller wants no pooled output
  int32_t* gather_src;    // [n_kv_heads * total_tokens] per packed row: token * n_kv_heads + head of its source
  int32_t* dev_flags;     // [8] scratch words (timeouts etc.)
  float* win_m;           // [n_seg][R] row statistics over the window keys (SLKV_ALL_CAUSAL without lse_opt)
  float* win_z;
  const float* lse_opt;   // the caller's row log-sum-exps, or null
  int max_score_ctas;     // > 0: the score kernels use at most this many CTAs (SMs); 0 = all
};

// kernel ids for launch accounting / per-kernel timing
enum KernelId { KID_SETUP = 0, KID_SCORE_LSE, KID_SCORE_VOTE, KID_POOL, KID_SELECT, KID_GATHER, KID_ALLOC, KID_SCORE_FUSED, KID_SCORE_PIPE, KID_WINDOW_STATS, KID_MERGE_LSE, KID_BEHAVIOR, KID_CP, KID_COUNT };

// Brackets one kernel launch: counts it and, when per-kernel timing is on for this thread, records a
// CUDA event pair around it on the launch stream.
struct LaunchScope {
  LaunchScope(int kid, cudaStream_t st, int* launches);
  ~LaunchScope();
  int kid_; cudaStream_t st_; int slot_;
};

// slkv_score's host-side argument checks, without a workspace: SLKV_OK or the status slkv_score would return
int check_score_args(const slkv_params* p, const void* q_win, const void* k, const int32_t* cu_seqlens_dev,
                     const int32_t* cu_seqlens_host, const float* pooled);

// host-side launchers; each returns a cudaError_t and adds to *launches
cudaError_t launch_alloc(const float* inf, int n_layers, int n_heads, int fixed, long long total, int within_layer,
                         int paper_rounding, long long cap, int32_t* budgets, int32_t* status, cudaStream_t st);
cudaError_t launch_behavior(const float* attn, long long row_stride, int row_len, long long n_rows,
                            const int32_t* needle_idx, int n_needle, long long needle_stride, const int32_t* topk_idx,
                            int n_topk, long long topk_stride, float* sf, float* lg, float* inf, cudaStream_t st);
// context-parallel selection (slkv_cp.cu)
cudaError_t launch_cp_merge_lse(const float* parts, int n_parts, long long n, float to_log2, float* out,
                                cudaStream_t st, int* launches);
cudaError_t launch_cp_need_init(const int32_t* budgets, int n_kv_heads, int window, long long seq_len, unsigned* prefix,
                                int32_t* need, cudaStream_t st, int* launches);
cudaError_t launch_cp_histogram(const float* pooled, int n_kv_heads, long long row_stride, int own_begin, int own_count,
                                int level, const unsigned* prefix, int32_t* hist, cudaStream_t st, int* launches);
cudaError_t launch_cp_descend(const int32_t* hist, int n_kv_heads, int level, unsigned* prefix, int32_t* need,
                              cudaStream_t st, int* launches);
cudaError_t launch_cp_local_ties(const int32_t* hist_local, const unsigned* prefix, int n_kv_heads, int32_t* ties,
                                 cudaStream_t st, int* launches);
cudaError_t launch_cp_emit(const float* pooled, long long row_stride, int own_begin, int own_count, long long pos0,
                           const unsigned* threshold, const int32_t* need, const int32_t* ties_all, int n_kv_heads,
                           int part, int window_rows, long long window_row0, long long window_pos0, long long capacity,
                           int32_t* offsets, int32_t* kept_idx, int32_t* gather_src, int32_t* rows, int32_t* take,
                           int32_t* cnt_gt, int32_t* cnt_eq, int32_t* status, cudaStream_t st, int* launches);
int cp_slices(int own_count);            // CTAs per head of the counting and packing kernels
cudaError_t launch_setup(const Problem& pb, const int32_t* budgets, int32_t* offsets, int64_t capacity,
                         int32_t* status, cudaStream_t st, int* launches);
int simt_chunk_keys();
size_t simt_smem_bytes(const Problem& pb);
// passes: 1 = row statistics only, 2 = votes only (the log-sum-exps come from lse_source_of), 3 = both
cudaError_t launch_score_simt(const Problem& pb, int passes, cudaStream_t st, int* launches);
// Row statistics of the window keys each window row sees causally (SLKV_ALL_CAUSAL) -> pb.win_m / pb.win_z, rows in
// the order of the score path (head_inner: r = i*G + hh).
cudaError_t launch_window_stats(const Problem& pb, bool head_inner, cudaStream_t st, int* launches);
// Merges the per-chunk (SIMT layout) or per-CTA (tensor layout, schedule in `plan`) row statistics and the window
// statistics, if any, into lse_out[n_seqs][n_q_heads][window] in the problem's lse_units.
cudaError_t launch_merge_lse_simt(const Problem& pb, float* lse_out, cudaStream_t st, int* launches);
cudaError_t launch_merge_lse_tensor(const Problem& pb, const int32_t* cu_host, float* lse_out, cudaStream_t st,
                                    int* launches);
LseSource lse_source_of(const Problem& pb);
float lse_out_scale(const Problem& pb);          // log2 units -> the problem's lse_units
bool tensor_q_head_inner(const slkv_params& p);
bool tensor_path_supported(const slkv_params& p);
int tensor_slot_stride(const Problem& pb);
void set_tensor_trace(void* dev_buf, size_t bytes);
// passes as launch_score_simt
cudaError_t launch_score_tensor(const Problem& pb, const int32_t* cu_host, int32_t* status, int passes,
                                cudaStream_t st, int* launches);
cudaError_t launch_pool(const Problem& pb, float* pooled, cudaStream_t st, int* launches);
cudaError_t launch_select(const Problem& pb, const float* pooled, const int32_t* budgets, const int32_t* offsets,
                          int32_t* kept_idx, int64_t capacity, cudaStream_t st, int* launches);
bool select_cta_supported(const Problem& pb);
cudaError_t launch_select_cta(const Problem& pb, float* pooled_out, const int32_t* budgets, int32_t* offsets,
                              int32_t* kept_idx, int64_t capacity, int32_t* status, cudaStream_t st, int* launches);
bool select_cluster_supported(const Problem& pb);
cudaError_t launch_select_cluster(const Problem& pb, float* pooled_out, const int32_t* budgets, int32_t* offsets,
                                  int32_t* kept_idx, int64_t capacity, int32_t* status, cudaStream_t st,
                                  int* launches);
// block_threads: 256, or 128 where the gather shares its SMs with a kernel that leaves few registers
cudaError_t launch_gather(const Problem& pb, const int32_t* offsets, const int32_t* kept_idx, void* k_out,
                          void* v_out, int64_t capacity, cudaStream_t st, int* launches, int block_threads = 256);

// ---- tensor-core score kernels: arguments and launch plans ---------------------------------------------------
struct TcArgs {
  SeqTables tab;
  float* part_m;
  float* part_z;
  float* vote;
  LseSource lse;
  int32_t* status;
  unsigned long long* trace;    // optional timeline buffer: kTraceSlots timestamps (ns) per CTA, or null
  int n_seqs, n_kv_heads, G, window, R, MT, n_stages, slot_stride, tiles_per_cta, total_tiles, barrier_slot;
  int fresh_inputs;             // vote pass only: no kernel of this library has read Q and K before this launch
  int barrier_extra;            // 0; 1 makes the grid-wide wait expect an arrival that never comes (diagnostics)
  int q_head_inner, k_head_inner;   // tensor-map dimension order: 1 = the head axis comes before the row axis
  float scale_log2;
};

// One layer's score problem, ready to launch: tensor maps of Q_win and K, kernel arguments, grid size.
struct TcPlan {
  CUtensorMap tm_q, tm_k;
  TcArgs a;
  int n_cta;
};
// Fills a plan (tensor maps, schedule, arguments) for a problem whose workspace is bound; n_cta = 0 when there is
// no history to score.  cudaErrorNotSupported when the driver has no tensor-map encoder.
cudaError_t plan_score_tensor(const Problem& pb, const int32_t* cu_host, int32_t* status, TcPlan* plan);
// Timeline buffer of this thread (diagnostics), or null: half 0 / 1, kTraceSlots words per CTA.
unsigned long long* tensor_trace_buffer(int half, int n_cta);
// Diagnostics: arm / consume the one-shot switch that makes the next inter-CTA wait of this thread's launches run out.
void expire_next_wait(int on);
int take_expire_next_wait();

// Several layers per launch, pass 1 of one layer beside pass 2 of the layer before: pass 1 of a[0..n_a), pass 2 of
// `pending` (pass 1 done by an earlier launch; may be null) and of a[0..n_a-1), or of all of a[] when `finish`.
// All plans share one shape.  The shapes it takes:
bool score_pipe_supported(const Problem& pb);
constexpr int kPipeMaxLayers = 8;
// votes_only: every plan carries the caller's row statistics, so both streams run pass 2 (no pending layer before or
// after the launch, no CTA waits for another).
cudaError_t launch_score_pipe(const TcPlan* pending, const TcPlan* const* a, int n_a, bool finish, bool votes_only,
                              cudaStream_t st, int* launches);

}  // namespace slkv
