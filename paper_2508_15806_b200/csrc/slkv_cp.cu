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
// A thread takes 16 consecutive positions and adds a run of equal digits at once: pooled scores come in runs (a
// maximum holds for pool_kernel positions), and neighbouring threads adding to the same bin one by one serialise.
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
  for (long long j0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 16; j0 < own_count;
       j0 += (long long)gridDim.x * blockDim.x * 16) {
    int run_digit = -1, run = 0;
#pragma unroll
    for (int q = 0; q < 16; ++q) {
      int dg = -1;
      if (j0 + q < own_count) {
        const unsigned bits = row[j0 + q];
        if (cp_match(bits, pf, level)) dg = (int)cp_digit(bits, level);
      }
      if (dg != run_digit) {
        if (run_digit >= 0) atomicAdd(&sh[run_digit], run);
        run_digit = dg; run = 0;
      }
      ++run;
    }
    if (run_digit >= 0) atomicAdd(&sh[run_digit], run);
  }
  __syncthreads();
  for (int b = threadIdx.x; b < kCpBins; b += blockDim.x)
    if (sh[b]) atomicAdd(&hist[h * kCpBins + b], sh[b]);
}

// One level of the descent on the histogram summed over all ranks: the digit d with
// count(digits > d) < need <= count(digits >= d) joins the prefix, need drops by the count above it (d = 0 if the counts
// above it never reach need).  need == 0: the prefix becomes all ones (nothing lies above it) and stays.
// One CTA of 256 threads per head; thread t holds the 8 digits 8t .. 8t+7 counted from the top.
__global__ void __launch_bounds__(256)
k_cp_descend(const int32_t* __restrict__ hist, int level, unsigned* __restrict__ prefix, int32_t* __restrict__ need) {
  __shared__ long long wtot[8];
  __shared__ int sh_found;
  pdl_launch_dependents();
  pdl_wait();
  const int h = blockIdx.x, t = threadIdx.x, lane = t & 31, wid = t >> 5;
  const int nd = need[h];
  if (nd <= 0) {
    if (t == 0) { prefix[h] = 0xffffffffu; need[h] = 0; }
    return;
  }
  const int bins = level == 2 ? 1024 : kCpBins;
  const int shift = level == 0 ? 21 : (level == 1 ? 10 : 0);
  if (t == 0) sh_found = 0;
  int c[8];
  long long s = 0;
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const int d = bins - 1 - (8 * t + q);
    c[q] = d >= 1 ? hist[h * kCpBins + d] : 0;           // digit 0 is where the search ends anyway
    s += c[q];
  }
  long long inc = s;
  for (int o = 1; o < 32; o <<= 1) {
    const long long n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (lane == 31) wtot[wid] = inc;
  __syncthreads();
  long long above = inc - s;
  for (int w2 = 0; w2 < wid; ++w2) above += wtot[w2];
  if (above < nd && above + s >= nd) {                   // the digit lies among this thread's eight
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      if (above + c[q] >= nd) {
        prefix[h] |= (unsigned)(bins - 1 - (8 * t + q)) << shift;
        need[h] = (int32_t)(nd - above);
        sh_found = 1;
        break;
      }
      above += c[q];
    }
  }
  __syncthreads();
  if (t == 0 && !sh_found) {                             // the counts above digit 0 do not reach need: digit 0
    long long total = 0;
    for (int w2 = 0; w2 < 8; ++w2) total += wtot[w2];
    need[h] = (int32_t)(nd - total);
  }
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

constexpr int kCpSlice = kCpThreads * kCpItems;       // positions per CTA of k_cp_count / k_cp_emit

// cnt_gt / cnt_eq[h][blk] = positions of slice blk of head h's owned range above / at the threshold.
__global__ void __launch_bounds__(kCpThreads)
k_cp_count(const float* __restrict__ pooled, long long row_stride, int own_begin, int own_count,
           const unsigned* __restrict__ threshold, int n_blk, int32_t* __restrict__ cnt_gt, int32_t* __restrict__ cnt_eq) {
  __shared__ int red[kCpThreads / 32];
  pdl_launch_dependents();
  pdl_wait();
  const int h = blockIdx.y, blk = blockIdx.x;
  const unsigned tau = threshold[h];
  const unsigned* row = reinterpret_cast<const unsigned*>(pooled + (long long)h * row_stride + own_begin);
  const long long first = (long long)blk * kCpSlice + threadIdx.x * kCpItems;
  int gt = 0, eq = 0;
#pragma unroll
  for (int q = 0; q < kCpItems; ++q)
    if (first + q < own_count) {
      const unsigned bits = row[first + q];
      gt += bits > tau;
      eq += bits == tau;
    }
  gt = cp_block_sum(gt, red);
  eq = cp_block_sum(eq, red);
  if (threadIdx.x == 0) { cnt_gt[h * n_blk + blk] = gt; cnt_eq[h * n_blk + blk] = eq; }
}

// Per head (one thread each): take[h] = its share of the ties = need[h] less the ties of the ranks before this one,
// within [0, own ties]; rows[h] = scores above the threshold + take + window rows; the counts become exclusive prefixes
// over the slices.  Then offsets = exclusive prefix of rows[] (thread 0).
__global__ void k_cp_plan(const int32_t* __restrict__ need, const int32_t* __restrict__ ties_all, int n_kv_heads, int part,
                          int window_rows, int n_blk, int32_t* __restrict__ cnt_gt, int32_t* __restrict__ cnt_eq,
                          int32_t* __restrict__ rows, int32_t* __restrict__ take, long long capacity,
                          int32_t* __restrict__ offsets, int32_t* __restrict__ status) {
  pdl_launch_dependents();
  pdl_wait();
  for (int h = threadIdx.x; h < n_kv_heads; h += blockDim.x) {
    int gt = 0, eq = 0;
    for (int b = 0; b < n_blk; ++b) {
      const int g = cnt_gt[h * n_blk + b], e = cnt_eq[h * n_blk + b];
      cnt_gt[h * n_blk + b] = gt; cnt_eq[h * n_blk + b] = eq;
      gt += g; eq += e;
    }
    long long before = 0;
    for (int r = 0; r < part; ++r) before += ties_all[r * n_kv_heads + h];
    long long t = (long long)need[h] - before;
    t = t < 0 ? 0 : (t > eq ? eq : t);
    take[h] = (int32_t)t;
    rows[h] = gt + (int32_t)t + window_rows;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    long long o = 0;
    for (int h = 0; h < n_kv_heads; ++h) { offsets[h] = (int32_t)o; o += rows[h]; }
    offsets[n_kv_heads] = (int32_t)o;
    if (o > capacity && status) atomicCAS(status, 0, (int)SLKV_ERR_CAPACITY);
  }
}

// Packs slice blk of head h's kept positions in ascending order: kept_idx = position in the whole sequence,
// gather_src = row of this rank's K / V (token * n_kv_heads + head); slice 0 also writes the window rows on the rank
// that holds them.  A kept position's packed row = offsets[h] + (scores above the threshold before it) +
// min(ties before it, take).
__global__ void __launch_bounds__(kCpThreads)
k_cp_emit(const float* __restrict__ pooled, long long row_stride, int own_begin, int own_count, long long pos0,
          const unsigned* __restrict__ threshold, const int32_t* __restrict__ rows, const int32_t* __restrict__ take,
          const int32_t* __restrict__ cnt_gt, const int32_t* __restrict__ cnt_eq, int n_blk, int n_kv_heads,
          int window_rows, long long window_row0, long long window_pos0, long long capacity,
          const int32_t* __restrict__ offsets, int32_t* __restrict__ kept_idx, int32_t* __restrict__ gather_src) {
  __shared__ unsigned wtot[kCpThreads / 32];
  pdl_launch_dependents();
  pdl_wait();
  const int h = blockIdx.y, blk = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const long long out0 = offsets[h];
  const unsigned tau = threshold[h];
  const int tk = take[h];
  const unsigned* row = reinterpret_cast<const unsigned*>(pooled + (long long)h * row_stride + own_begin);
  const long long first = (long long)blk * kCpSlice + tid * kCpItems;
  unsigned bits[kCpItems];
  unsigned packed = 0;                           // ties in the high half, scores above the threshold in the low half
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
  if (lane == 31) wtot[wid] = inc;
  __syncthreads();
  if (wid == 0) {
    unsigned w = wtot[lane], winc = w;
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned n = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += n;
    }
    wtot[lane] = winc - w;                       // exclusive over the warps
  }
  __syncthreads();
  const unsigned excl = wtot[wid] + inc - packed;
  unsigned gb = (unsigned)cnt_gt[h * n_blk + blk] + (excl & 65535u), eb = (unsigned)cnt_eq[h * n_blk + blk] + (excl >> 16);
#pragma unroll
  for (int q = 0; q < kCpItems; ++q) {
    if (first + q >= own_count) break;
    const bool gt = bits[q] > tau, eq = bits[q] == tau;
    if (gt || (eq && (int)eb < tk)) {
      const long long o = out0 + gb + min(eb, (unsigned)tk);
      if (o < capacity) {
        kept_idx[o] = (int32_t)(pos0 + first + q);
        gather_src[o] = (int32_t)((own_begin + first + q) * n_kv_heads + h);
      }
    }
    gb += gt;
    eb += eq;
  }
  // window rows (Algorithm 3 l.4, l.10): always kept, behind the history rows, on the rank that holds them
  if (blk == 0) {
    const long long w0 = out0 + rows[h] - window_rows;
    for (int i = tid; i < window_rows; i += kCpThreads)
      if (w0 + i < capacity) {
        kept_idx[w0 + i] = (int32_t)(window_pos0 + i);
        gather_src[w0 + i] = (int32_t)((window_row0 + i) * n_kv_heads + h);
      }
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
  return launch_pdl(k_cp_descend, dim3(n_kv_heads), dim3(256), 0, st, 1, hist, level, prefix, need);
}

cudaError_t launch_cp_local_ties(const int32_t* hist_local, const unsigned* prefix, int n_kv_heads, int32_t* ties,
                                 cudaStream_t st, int* launches) {
  LaunchScope scope(KID_CP, st, launches);
  return launch_pdl(k_cp_local_ties, dim3((n_kv_heads + 127) / 128), dim3(128), 0, st, 1, hist_local, prefix,
                    n_kv_heads, ties);
}

int cp_slices(int own_count) { return own_count > 0 ? (own_count + kCpSlice - 1) / kCpSlice : 1; }

cudaError_t launch_cp_emit(const float* pooled, long long row_stride, int own_begin, int own_count, long long pos0,
                           const unsigned* threshold, const int32_t* need, const int32_t* ties_all, int n_kv_heads,
                           int part, int window_rows, long long window_row0, long long window_pos0, long long capacity,
                           int32_t* offsets, int32_t* kept_idx, int32_t* gather_src, int32_t* rows, int32_t* take,
                           int32_t* cnt_gt, int32_t* cnt_eq, int32_t* status, cudaStream_t st, int* launches) {
  const int n_blk = cp_slices(own_count);
  {
    LaunchScope scope(KID_CP, st, launches);
    cudaError_t e = launch_pdl(k_cp_count, dim3(n_blk, n_kv_heads), dim3(kCpThreads), 0, st, 1, pooled, row_stride,
                               own_begin, own_count, threshold, n_blk, cnt_gt, cnt_eq);
    if (e != cudaSuccess) return e;
  }
  {
    LaunchScope scope(KID_CP, st, launches);
    cudaError_t e = launch_pdl(k_cp_plan, dim3(1), dim3(256), 0, st, 1, need, ties_all, n_kv_heads, part, window_rows,
                               n_blk, cnt_gt, cnt_eq, rows, take, capacity, offsets, status);
    if (e != cudaSuccess) return e;
  }
  LaunchScope scope(KID_CP, st, launches);
  return launch_pdl(k_cp_emit, dim3(n_blk, n_kv_heads), dim3(kCpThreads), 0, st, 1, pooled, row_stride, own_begin,
                    own_count, pos0, threshold, (const int32_t*)rows, (const int32_t*)take, (const int32_t*)cnt_gt,
                    (const int32_t*)cnt_eq, n_blk, n_kv_heads, window_rows, window_row0, window_pos0, capacity,
                    (const int32_t*)offsets, kept_idx, gather_src);
}

}  // namespace slkv
