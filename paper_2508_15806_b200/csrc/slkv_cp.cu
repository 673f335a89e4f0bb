// Context-parallel selection (Sec. 3.4, Eq. 8; Algorithm 3 with one sequence's history keys split over ranks).
//
// Each rank holds a contiguous range of the history keys (plus pool_kernel / 2 rows of its neighbours' on each side, so
// that pooling needs nothing from them) and scores it with the ordinary score kernels against row log-sum-exps merged
// over all ranks.  What is left is one top-k per KV head over scores that live on different ranks: a radix descent over
// the scores' bit patterns (11 + 11 + 10 bits) whose histograms are summed across ranks between the levels, the ties at
// the threshold handed out in rank order (lower positions first, as on one GPU), then every rank packs the rows it owns.
// Integer counters only: the kept set does not depend on timing or on the number of ranks.
#include "slkv_internal.cuh"

namespace slkv {
namespace {

constexpr int kCpBins = 2048;
constexpr int kCpThreads = 1024;
constexpr int kCpItems = 4;                 // consecutive positions per thread and round of k_cp_emit

__device__ __forceinline__ unsigned cp_digit(unsigned bits, int level) {
  return level == 0 ? bits >> 21 : (level == 1 ? (bits >> 10) & 2047u : bits & 1023u);
}
__device__ __forceinline__ bool cp_match(unsigned bits, unsigned prefix, int level) {
  return level == 0 || (level == 1 ? (bits >> 21) == (prefix >> 21) : (bits >> 10) == (prefix >> 10));
}

// lse_out[i] = log-sum-exp over the parts of lse_parts[r][i], all in the units `to_log2` converts to base 2.
__global__ void k_cp_merge_lse(const float* __restrict__ parts, int n_parts, long long n, float to_log2,
                               float* __restrict__ out) {
  pdl_launch_dependents();
  pdl_wait();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float m = -INFINITY;
  for (int r = 0; r < n_parts; ++r) m = fmaxf(m, parts[(long long)r * n + i] * to_log2);
  if (!(m > -INFINITY)) { out[i] = -INFINITY; return; }       // no rank has a key for this row
  float z = 0.f;
  for (int r = 0; r < n_parts; ++r) z += exp2f(parts[(long long)r * n + i] * to_log2 - m);
  out[i] = (m + log2f(z)) / to_log2;
}

// need[h] = history rows head h keeps of the whole sequence (Algorithm 3 l.1-3, l.7), prefix[h] = 0.
__global__ void k_cp_need_init(const int32_t* __restrict__ budgets, int n_kv_heads, int window, long long seq_len,
                               unsigned* __restrict__ prefix, int32_t* __restrict__ need) {
  pdl_launch_dependents();
  pdl_wait();
  const int h = blockIdx.x * blockDim.x + threadIdx.x;
  if (h >= n_kv_heads) return;
  const long long c = max((long long)budgets[h], (long long)window);
  const long long kept = min(seq_len, c);
  need[h] = (int32_t)(kept - min(seq_len, (long long)window));
  prefix[h] = 0u;
}

// hist[h][d] += own positions of head h whose bits agree with prefix[h] above this level's digit and have digit d.
__global__ void __launch_bounds__(256)
k_cp_histogram(const float* __restrict__ pooled, long long row_stride, int own_begin, int own_count, int level,
               const unsigned* __restrict__ prefix, int32_t* __restrict__ hist) {
  __shared__ int sh[kCpBins];
  pdl_launch_dependents();
  const int h = blockIdx.y;
  for (int b = threadIdx.x; b < kCpBins; b += blockDim.x) sh[b] = 0;
  pdl_wait();
  __syncthreads();
  const unsigned pf = prefix[h];
  const unsigned* row = reinterpret_cast<const unsigned*>(pooled + (long long)h * row_stride + own_begin);
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < own_count; j += gridDim.x * blockDim.x) {
    const unsigned bits = row[j];
    if (cp_match(bits, pf, level)) atomicAdd(&sh[cp_digit(bits, level)], 1);
  }
  __syncthreads();
  for (int b = threadIdx.x; b < kCpBins; b += blockDim.x)
    if (sh[b]) atomicAdd(&hist[h * kCpBins + b], sh[b]);
}

// One level of the descent on the histogram summed over all ranks: the digit d with
// count(digits > d) < need <= count(digits >= d) joins the prefix, need drops by the count above it.
// need == 0: the prefix becomes all ones (nothing lies above it) and stays.
__global__ void k_cp_descend(const int32_t* __restrict__ hist, int n_kv_heads, int level, unsigned* __restrict__ prefix,
                             int32_t* __restrict__ need) {
  pdl_launch_dependents();
  pdl_wait();
  const int h = blockIdx.x * blockDim.x + threadIdx.x;
  if (h >= n_kv_heads) return;
  const int nd = need[h];
  if (nd <= 0) { prefix[h] = 0xffffffffu; need[h] = 0; return; }
  const int bins = level == 2 ? 1024 : kCpBins;
  const int shift = level == 0 ? 21 : (level == 1 ? 10 : 0);
  long long above = 0;
  int d = bins - 1;
  for (; d > 0; --d) {
    const int c = hist[h * kCpBins + d];
    if (above + c >= nd) break;
    above += c;
  }
  prefix[h] |= (unsigned)d << shift;
  need[h] = (int32_t)(nd - above);
}

// ties[h] = this rank's positions whose score equals the threshold = its last-level histogram at the threshold's digit.
__global__ void k_cp_local_ties(const int32_t* __restrict__ hist_local, const unsigned* __restrict__ prefix,
                                int n_kv_heads, int32_t* __restrict__ ties) {
  pdl_launch_dependents();
  pdl_wait();
  const int h = blockIdx.x * blockDim.x + threadIdx.x;
  if (h >= n_kv_heads) return;
  ties[h] = prefix[h] == 0xffffffffu ? 0 : hist_local[h * kCpBins + (prefix[h] & 1023u)];
}

__device__ __forceinline__ int cp_block_sum(int v, int* red) {
  __syncthreads();
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  int t = 0;
  for (int w = 0; w < kCpThreads / 32; ++w) t += red[w];
  return t;
}

// rows[h] = packed rows this rank writes for head h: scores above the threshold, its share of the ties, its window
// rows; take[h] = that share: need[h] less the ties of the ranks before this one, within [0, own ties].
__global__ void __launch_bounds__(kCpThreads)
k_cp_count(const float* __restrict__ pooled, long long row_stride, int own_begin, int own_count,
           const unsigned* __restrict__ threshold, const int32_t* __restrict__ need,
           const int32_t* __restrict__ ties_all, int n_kv_heads, int part, int window_rows,
           int32_t* __restrict__ rows, int32_t* __restrict__ take) {
  __shared__ int red[kCpThreads / 32];
  pdl_launch_dependents();
  pdl_wait();
  const int h = blockIdx.x;
  const unsigned tau = threshold[h];
  const unsigned* row = reinterpret_cast<const unsigned*>(pooled + (long long)h * row_stride + own_begin);
  int gt = 0, eq = 0;
  for (int j = threadIdx.x; j < own_count; j += kCpThreads) {
    const unsigned bits = row[j];
    gt += bits > tau;
    eq += bits == tau;
  }
  gt = cp_block_sum(gt, red);
  eq = cp_block_sum(eq, red);
  if (threadIdx.x == 0) {
    long long before = 0;
    for (int r = 0; r < part; ++r) before += ties_all[r * n_kv_heads + h];
    long long t = (long long)need[h] - before;
    t = t < 0 ? 0 : (t > eq ? eq : t);
    take[h] = (int32_t)t;
    rows[h] = gt + (int32_t)t + window_rows;
  }
}

// Packs head h's kept positions in ascending order: kept_idx = position in the whole sequence, gather_src = row of this
// rank's K / V (token * n_kv_heads + head); then the window rows on the rank that holds them; offsets = exclusive
// prefix of rows[].  A kept position's packed row = (scores above the threshold before it) + min(ties before it, take).
__global__ void __launch_bounds__(kCpThreads)
k_cp_emit(const float* __restrict__ pooled, long long row_stride, int own_begin, int own_count, long long pos0,
          const unsigned* __restrict__ threshold, const int32_t* __restrict__ rows, const int32_t* __restrict__ take,
          int n_kv_heads, int window_rows, long long window_row0, long long window_pos0, long long capacity,
          int32_t* __restrict__ offsets, int32_t* __restrict__ kept_idx, int32_t* __restrict__ gather_src,
          int32_t* __restrict__ status) {
  __shared__ unsigned wtot[kCpThreads / 32];
  __shared__ unsigned sh_base;
  pdl_launch_dependents();
  pdl_wait();
  const int h = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  long long out0 = 0;
  for (int g = 0; g < h; ++g) out0 += rows[g];
  if (tid == 0) {
    offsets[h] = (int32_t)out0;
    if (h == n_kv_heads - 1) {
      offsets[n_kv_heads] = (int32_t)(out0 + rows[h]);
      if (out0 + rows[h] > capacity && status) atomicCAS(status, 0, (int)SLKV_ERR_CAPACITY);
    }
  }
  const unsigned tau = threshold[h];
  const int tk = take[h];
  const unsigned* row = reinterpret_cast<const unsigned*>(pooled + (long long)h * row_stride + own_begin);
  unsigned g_run = 0, e_run = 0;                 // kept-above and tie counts of the rounds before
  for (int j0 = 0; j0 < own_count; j0 += kCpThreads * kCpItems) {
    const int first = j0 + tid * kCpItems;
    unsigned bits[kCpItems];
    unsigned packed = 0;                         // ties in the high half, scores above the threshold in the low half
#pragma unroll
    for (int q = 0; q < kCpItems; ++q) {
      bits[q] = first + q < own_count ? row[first + q] : 0u;
      if (first + q < own_count) packed += (bits[q] > tau ? 1u : 0u) + (bits[q] == tau ? 65536u : 0u);
    }
    unsigned inc = packed;
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned n = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += n;
    }
    __syncthreads();                             // wtot / sh_base of the round before are read
    if (lane == 31) wtot[wid] = inc;
    __syncthreads();
    if (wid == 0) {
      unsigned w = wtot[lane], winc = w;
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned n = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += n;
      }
      wtot[lane] = winc - w;                     // exclusive over the warps
      if (lane == 31) sh_base = winc;            // the round's totals
    }
    __syncthreads();
    const unsigned excl = wtot[wid] + inc - packed;
    unsigned gb = g_run + (excl & 65535u), eb = e_run + (excl >> 16);
#pragma unroll
    for (int q = 0; q < kCpItems; ++q) {
      if (first + q >= own_count) break;
      const bool gt = bits[q] > tau, eq = bits[q] == tau;
      if (gt || (eq && (int)eb < tk)) {
        const long long o = out0 + gb + min(eb, (unsigned)tk);
        if (o < capacity) {
          kept_idx[o] = (int32_t)(pos0 + first + q);
          gather_src[o] = (int32_t)((long long)(own_begin + first + q) * n_kv_heads + h);
        }
      }
      gb += gt;
      eb += eq;
    }
    g_run += sh_base & 65535u;
    e_run += sh_base >> 16;
  }
  // window rows (Algorithm 3 l.4, l.10): always kept, behind the history rows, on the rank that holds them
  const long long w0 = out0 + rows[h] - window_rows;
  for (int i = tid; i < window_rows; i += kCpThreads)
    if (w0 + i < capacity) {
      kept_idx[w0 + i] = (int32_t)(window_pos0 + i);
      gather_src[w0 + i] = (int32_t)((window_row0 + i) * n_kv_heads + h);
    }
}

}  // namespace

cudaError_t launch_cp_merge_lse(const float* parts, int n_parts, long long n, float to_log2, float* out,
                                cudaStream_t st, int* launches) {
  LaunchScope scope(KID_CP, st, launches);
  return launch_pdl(k_cp_merge_lse, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st, 1, parts, n_parts, n, to_log2, out);
}

cudaError_t launch_cp_need_init(const int32_t* budgets, int n_kv_heads, int window, long long seq_len, unsigned* prefix,
                                int32_t* need, cudaStream_t st, int* launches) {
  LaunchScope scope(KID_CP, st, launches);
  return launch_pdl(k_cp_need_init, dim3((n_kv_heads + 127) / 128), dim3(128), 0, st, 1, budgets, n_kv_heads, window,
                    seq_len, prefix, need);
}

cudaError_t launch_cp_histogram(const float* pooled, int n_kv_heads, long long row_stride, int own_begin, int own_count,
                                int level, const unsigned* prefix, int32_t* hist, cudaStream_t st, int* launches) {
  cudaError_t e = cudaMemsetAsync(hist, 0, (size_t)n_kv_heads * kCpBins * sizeof(int32_t), st);
  if (e != cudaSuccess) return e;
  int bx = (own_count + 256 * 16 - 1) / (256 * 16);
  bx = bx < 1 ? 1 : (bx > 64 ? 64 : bx);
  LaunchScope scope(KID_CP, st, launches);
  return launch_pdl(k_cp_histogram, dim3(bx, n_kv_heads), dim3(256), 0, st, 1, pooled, row_stride, own_begin, own_count,
                    level, prefix, hist);
}

cudaError_t launch_cp_descend(const int32_t* hist, int n_kv_heads, int level, unsigned* prefix, int32_t* need,
                              cudaStream_t st, int* launches) {
  LaunchScope scope(KID_CP, st, launches);
  return launch_pdl(k_cp_descend, dim3((n_kv_heads + 127) / 128), dim3(128), 0, st, 1, hist, n_kv_heads, level, prefix,
                    need);
}

cudaError_t launch_cp_local_ties(const int32_t* hist_local, const unsigned* prefix, int n_kv_heads, int32_t* ties,
                                 cudaStream_t st, int* launches) {
  LaunchScope scope(KID_CP, st, launches);
  return launch_pdl(k_cp_local_ties, dim3((n_kv_heads + 127) / 128), dim3(128), 0, st, 1, hist_local, prefix,
                    n_kv_heads, ties);
}

cudaError_t launch_cp_emit(const float* pooled, long long row_stride, int own_begin, int own_count, long long pos0,
                           const unsigned* threshold, const int32_t* need, const int32_t* ties_all, int n_kv_heads,
                           int part, int window_rows, long long window_row0, long long window_pos0, long long capacity,
                           int32_t* offsets, int32_t* kept_idx, int32_t* gather_src, int32_t* rows, int32_t* take,
                           int32_t* status, cudaStream_t st, int* launches) {
  {
    LaunchScope scope(KID_CP, st, launches);
    cudaError_t e = launch_pdl(k_cp_count, dim3(n_kv_heads), dim3(kCpThreads), 0, st, 1, pooled, row_stride, own_begin,
                               own_count, threshold, need, ties_all, n_kv_heads, part, window_rows, rows, take);
    if (e != cudaSuccess) return e;
  }
  LaunchScope scope(KID_CP, st, launches);
  return launch_pdl(k_cp_emit, dim3(n_kv_heads), dim3(kCpThreads), 0, st, 1, pooled, row_stride, own_begin, own_count,
                    pos0, threshold, (const int32_t*)rows, (const int32_t*)take, n_kv_heads, window_rows, window_row0,
                    window_pos0, capacity, offsets, kept_idx, gather_src, status);
}

}  // namespace slkv
