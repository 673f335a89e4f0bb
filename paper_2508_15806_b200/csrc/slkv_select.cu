// Sequence tables, pooling, per-head variable-k selection and the packed K/V gather
// (Sec. 3.4, Eq. 8; Algorithm 3 lines 1-4 and 7-10).
#include "slkv_internal.cuh"

namespace slkv {
namespace {

constexpr int kScanThreads = 1024;

// Exclusive scan of one value per thread across the CTA; returns the exclusive prefix, *total = CTA sum.
template <typename T>
__device__ __forceinline__ T block_excl_scan(T v, T* warp_tot /*[32]*/, T* total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
  T inc = v;
  for (int o = 1; o < 32; o <<= 1) {
    T n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  __syncthreads();                       // warp_tot may still be read from a previous call
  if (lane == 31) warp_tot[wid] = inc;
  __syncthreads();
  T base = 0, tot = 0;
  for (int w = 0; w < nw; ++w) {
    T t = warp_tot[w];
    if (w < wid) base += t;
    tot += t;
  }
  *total = tot;
  return base + inc - v;
}

__device__ __forceinline__ int kept_rows(int len, int budget, int window) {
  // Algorithm 3 l.1-3 (keep all when the length fits the budget) and the always-kept window
  return min(len, max(budget, window));
}

// hist_off[s] = sum_{s'<s} max(len_s' - w, 0); with budgets: offsets[seg] = packed row where segment
// seg = s*Hkv + h starts.
__global__ void __launch_bounds__(kScanThreads, 1)
k_setup(const int32_t* __restrict__ cu, int n_seqs, int n_kv_heads, int window, const int32_t* __restrict__ budgets,
        int64_t* __restrict__ hist_off, int32_t* __restrict__ tile_off, int32_t* __restrict__ offsets,
        long long capacity, int32_t* __restrict__ status) {
  __shared__ long long wt[32];
  const int tid = threadIdx.x;
  pdl_launch_dependents();
  pdl_wait();
  long long run = 0, run_tiles = 0;
  for (int s0 = 0; s0 < n_seqs; s0 += kScanThreads) {
    int s = s0 + tid;
    long long nh = 0;
    if (s < n_seqs) nh = max(cu[s + 1] - cu[s] - window, 0);
    long long tot, ex = block_excl_scan<long long>(nh, wt, &tot);
    if (s < n_seqs) hist_off[s] = run + ex;
    run += tot;
    ex = block_excl_scan<long long>((nh + 127) >> 7, wt, &tot);     // 128-key tiles of the tensor-core path
    if (s < n_seqs) tile_off[s] = (int32_t)(run_tiles + ex);
    run_tiles += tot;
  }
  if (tid == 0) { hist_off[n_seqs] = run; tile_off[n_seqs] = (int32_t)run_tiles; }
  if (budgets == nullptr) return;
  const int n_seg = n_seqs * n_kv_heads;
  run = 0;
  for (int g0 = 0; g0 < n_seg; g0 += kScanThreads) {
    int seg = g0 + tid;
    long long kept = 0;
    if (seg < n_seg) {
      int s = seg / n_kv_heads, h = seg - s * n_kv_heads;
      kept = kept_rows(cu[s + 1] - cu[s], budgets[h], window);
    }
    long long tot, ex = block_excl_scan<long long>(kept, wt, &tot);
    if (seg < n_seg) offsets[seg] = (int32_t)(run + ex);
    run += tot;
  }
  if (tid == 0) {
    offsets[n_seg] = (int32_t)run;
    if (run > capacity && status) *status = SLKV_ERR_CAPACITY;
  }
}

// pooled[j] = max (or zero-padded mean) of vote[j-r .. j+r] inside the segment's history.
__global__ void __launch_bounds__(256)
k_pool(const float* __restrict__ vote, float* __restrict__ pooled, const __grid_constant__ SeqTables tab,
       int n_kv_heads, int window, int pool_kernel, int pool_mode) {
  pdl_launch_dependents();
  pdl_wait();
  const int s = blockIdx.z, h = blockIdx.y;
  const int n_hist = max(tab.cu_at(s + 1) - tab.cu_at(s) - window, 0);
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n_hist) return;
  const long long base = tab.hist_at(s) * n_kv_heads + (long long)h * n_hist;
  const float* src = vote + base;
  const int r = pool_kernel >> 1;
  const int lo = max(j - r, 0), hi = min(j + r, n_hist - 1);
  float acc;
  if (pool_mode == SLKV_POOL_MAX) {
    acc = src[lo];
    for (int t = lo + 1; t <= hi; ++t) acc = fmaxf(acc, src[t]);
  } else {
    acc = 0.f;
    for (int t = lo; t <= hi; ++t) acc += src[t];
    acc = acc / (float)pool_kernel;
  }
  pooled[base + j] = acc;
}

// One CTA per segment.  Finds the k-th largest pooled score by a 4 x 8-bit radix descent over the
// float bit patterns (scores are >= 0, so unsigned order = float order), then writes the positions of
// the k best in ascending order (equal scores: lower position first) followed by the window positions.
__global__ void __launch_bounds__(kScanThreads, 1)
k_select(const float* __restrict__ pooled, const __grid_constant__ SeqTables tab,
         const int32_t* __restrict__ budgets, const int32_t* __restrict__ offsets, int32_t* __restrict__ kept_idx,
         int32_t* __restrict__ gather_src, int n_kv_heads, int window, long long capacity) {
  __shared__ int hist[256];
  __shared__ int wt[32];
  __shared__ unsigned sh_prefix;
  __shared__ int sh_need;
  const int tid = threadIdx.x;
  pdl_launch_dependents();
  pdl_wait();
  const int seg = blockIdx.x;
  const int s = seg / n_kv_heads, h = seg - s * n_kv_heads;
  const int len = tab.cu_at(s + 1) - tab.cu_at(s);
  const int n_hist = max(len - window, 0);
  const int n_win = min(len, window);
  const int k = kept_rows(len, budgets[h], window) - n_win;      // history rows to keep (C_H = C - window)
  const long long out0 = offsets[seg];
  const int src_base = tab.cu_at(s) * n_kv_heads + h;           // source row of position j: src_base + j * n_kv_heads
  const unsigned* src = reinterpret_cast<const unsigned*>(pooled + tab.hist_at(s) * n_kv_heads + (long long)h * n_hist);

  // window rows (Algorithm 3 l.4, l.10): always kept, appended after the history rows
  for (int t = tid; t < n_win; t += kScanThreads) {
    long long o = out0 + k + t;
    if (o < capacity) {
      kept_idx[o] = len - n_win + t;
      gather_src[o] = src_base + (len - n_win + t) * n_kv_heads;
    }
  }
  if (k <= 0) return;
  if (k >= n_hist) {                                             // nothing to drop
    for (int j = tid; j < n_hist; j += kScanThreads)
      if (out0 + j < capacity) {
        kept_idx[out0 + j] = j;
        gather_src[out0 + j] = src_base + j * n_kv_heads;
      }
    return;
  }

  unsigned prefix = 0, mask = 0;
  int need = k;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int j = tid; j < n_hist; j += kScanThreads) {
      unsigned v = src[j];
      if ((v & mask) == prefix) atomicAdd(&hist[(v >> shift) & 255u], 1);
    }
    __syncthreads();
    if (tid == 0) {
      int cum = 0, b = 255;
      for (; b > 0; --b) {
        int c = hist[b];
        if (cum + c >= need) break;
        cum += c;
      }
      sh_prefix = prefix | ((unsigned)b << shift);
      sh_need = need - cum;
    }
    __syncthreads();
    prefix = sh_prefix;
    need = sh_need;
    mask |= 255u << shift;
    __syncthreads();
  }
  const unsigned tau = prefix;      // k-th largest value; `need` of the elements equal to it are kept

  int gt_seen = 0, eq_seen = 0;
  for (int j0 = 0; j0 < n_hist; j0 += kScanThreads) {
    const int j = j0 + tid;
    unsigned v = (j < n_hist) ? src[j] : 0u;
    const int gt = (j < n_hist) && (v > tau);
    const int eq = (j < n_hist) && (v == tau);
    int tot, ex = block_excl_scan<int>(gt | (eq << 16), wt, &tot);
    const int gt_before = gt_seen + (ex & 0xffff), eq_before = eq_seen + (ex >> 16);
    if (gt || (eq && eq_before < need)) {
      long long o = out0 + gt_before + min(eq_before, need);
      if (o < capacity) {
        kept_idx[o] = j;
        gather_src[o] = src_base + j * n_kv_heads;
      }
    }
    gt_seen += tot & 0xffff;
    eq_seen += tot >> 16;
  }
}

// Copies the kept rows of K and V into the packed cache: 16 bytes per lane, a row per lane group.  The
// selection kernel left the source row (token * n_kv_heads + head) of every packed row in gather_src, so a
// row costs two dependent memory round trips (source index, then the row itself).
__global__ void __launch_bounds__(256)
k_gather(const unsigned char* __restrict__ k, const unsigned char* __restrict__ v, unsigned char* __restrict__ k_out,
         unsigned char* __restrict__ v_out, const int32_t* __restrict__ offsets,
         const int32_t* __restrict__ gather_src, int n_seg, int n_kv_heads, int row_bytes, long long k_tok_bytes,
         long long k_head_bytes, long long v_tok_bytes, long long v_head_bytes, long long max_rows) {
  pdl_launch_dependents();
  const int lanes = row_bytes >> 4;                       // 16-byte lanes per row (power of two <= 32)
  const int rows_per_cta = blockDim.x / lanes;
  const int lane = threadIdx.x % lanes, sub = threadIdx.x / lanes;
  pdl_wait();
  const long long n_rows = min((long long)offsets[n_seg], max_rows);
  for (long long r = (long long)blockIdx.x * rows_per_cta + sub; r < max_rows;
       r += (long long)gridDim.x * rows_per_cta) {
    const int src = gather_src[r];                        // in bounds for r < max_rows; valid for r < n_rows
    if (r >= n_rows) break;
    const int tok = src / n_kv_heads, h = src - tok * n_kv_heads;
    const uint4 kv = *reinterpret_cast<const uint4*>(k + tok * k_tok_bytes + h * k_head_bytes + lane * 16);
    const uint4 vv = *reinterpret_cast<const uint4*>(v + tok * v_tok_bytes + h * v_head_bytes + lane * 16);
    *reinterpret_cast<uint4*>(k_out + r * row_bytes + lane * 16) = kv;
    *reinterpret_cast<uint4*>(v_out + r * row_bytes + lane * 16) = vv;
  }
}

}  // namespace

cudaError_t launch_setup(const Problem& pb, const int32_t* budgets, int32_t* offsets, int64_t capacity,
                         int32_t* status, cudaStream_t st, int* launches) {
  LaunchScope scope(KID_SETUP, st, launches);
  return launch_pdl(k_setup, dim3(1), dim3(kScanThreads), 0, st, 1, pb.cu, pb.p.n_seqs, pb.p.n_kv_heads,
                    pb.p.window, budgets, pb.hist_off, pb.tile_off, offsets, (long long)capacity, status);
}

cudaError_t launch_pool(const Problem& pb, float* pooled, cudaStream_t st, int* launches) {
  if (pb.max_hist <= 0) return cudaSuccess;
  dim3 grid((pb.max_hist + 255) / 256, pb.p.n_kv_heads, pb.p.n_seqs);
  LaunchScope scope(KID_POOL, st, launches);
  return launch_pdl(k_pool, grid, dim3(256), 0, st, 1, (const float*)pb.vote, pooled, pb.tab, pb.p.n_kv_heads,
                    pb.p.window, pb.p.pool_kernel, pb.p.pool_mode);
}

cudaError_t launch_select(const Problem& pb, const float* pooled, const int32_t* budgets, const int32_t* offsets,
                          int32_t* kept_idx, int64_t capacity, cudaStream_t st, int* launches) {
  LaunchScope scope(KID_SELECT, st, launches);
  return launch_pdl(k_select, dim3(pb.n_seg), dim3(kScanThreads), 0, st, 1, pooled, pb.tab, budgets, offsets,
                    kept_idx, pb.gather_src, pb.p.n_kv_heads, pb.p.window, (long long)capacity);
}

cudaError_t launch_gather(const Problem& pb, const int32_t* offsets, const int32_t* kept_idx, void* k_out,
                          void* v_out, int64_t capacity, cudaStream_t st, int* launches, int block_threads) {
  (void)kept_idx;
  const int row_bytes = pb.p.head_dim * pb.elem;
  if (block_threads != 128) block_threads = 256;
  const int rows_per_cta = block_threads / (row_bytes >> 4);
  long long max_rows = (long long)pb.p.n_kv_heads * pb.total_tokens;
  if (capacity < max_rows) max_rows = capacity;
  if (max_rows <= 0) return cudaSuccess;
  long long want = (max_rows + rows_per_cta - 1) / rows_per_cta;
  const int max_grid = 148 * 8 * (256 / block_threads);
  int grid = (int)(want < max_grid ? want : max_grid);
  LaunchScope scope(KID_GATHER, st, launches);
  return launch_pdl(k_gather, dim3(grid), dim3(block_threads), 0, st, 1, (const unsigned char*)pb.k,
                    (const unsigned char*)pb.v, (unsigned char*)k_out, (unsigned char*)v_out, offsets,
                    (const int32_t*)pb.gather_src, pb.n_seg, pb.p.n_kv_heads, row_bytes,
                    (long long)(pb.p.k_stride_tok * pb.elem), (long long)(pb.p.k_stride_head * pb.elem),
                    (long long)(pb.p.v_stride_tok * pb.elem), (long long)(pb.p.v_stride_head * pb.elem), max_rows);
}

}  // namespace slkv
