// Pooling + per-head variable-k selection, one CTA per (sequence, KV head) segment of up to 32768 history
// positions (Sec. 3.4, Eq. 8; Algorithm 3 lines 1-4, 7-8).
//
// A segment this size fits one CTA's registers: thread t owns the 32 consecutive positions [32t, 32t+32).
// The votes arrive with coalesced loads, pass once through (bank-conflict-free, padded) shared memory to reach
// their owners together with the pooling halo, and from then on the pooled scores live in registers.  The
// k-th largest is found by a radix descent over the float bit patterns (11 + 11 + 10 bits; scores are >= 0,
// so unsigned order = float order) with one shared-memory histogram per level; a thread feeds it one atomic
// per run of equal digits among its positions (max pooling makes neighbours equal).  No step leaves the CTA,
// so there is nothing to exchange between CTAs; integer counters only, so the result does not depend on timing.
#include "slkv_internal.cuh"

namespace slkv {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kItems = 32;                            // positions per thread
constexpr int kMaxHist = kThreads * kItems;           // 32768
constexpr int kBins = 2048;
constexpr int kMaxRadius = 4;                         // pool_kernel <= 9
// position i (shifted by one 32-block so that the left halo exists) -> padded shared-memory index
__device__ __forceinline__ int padded(int i) { return i + 32 + ((i + 32) >> 5); }
constexpr int kPaddedFloats = (kMaxHist + 64) + ((kMaxHist + 64) >> 5) + 1;

struct SelCtaArgs {
  const float* vote;
  float* pooled_out;          // optional
  const int32_t* budgets;
  int32_t* offsets;
  int32_t* kept_idx;
  int32_t* gather_src;        // per packed row: token * n_kv_heads + head of the source row
  int32_t* status;
  int n_seqs, n_kv_heads, window, pool_mode;
  long long capacity;
  SeqTables tab;
};

__device__ __forceinline__ int kept_rows(int len, int budget, int window) { return min(len, max(budget, window)); }

// Inclusive scan of one value per thread over the CTA in thread order; *total = CTA sum.  `wtot` is 32 words.
__device__ __forceinline__ unsigned block_incl_scan(unsigned v, unsigned* wtot, unsigned* total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  unsigned inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  __syncthreads();                       // wtot may still be read from an earlier call
  if (lane == 31) wtot[wid] = inc;
  __syncthreads();
  unsigned w = wtot[lane];               // every warp scans the 32 warp totals itself
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned n = __shfl_up_sync(0xffffffffu, w, o);
    if (lane >= o) w += n;
  }
  *total = __shfl_sync(0xffffffffu, w, 31);
  const unsigned before = __shfl_sync(0xffffffffu, w, max(wid - 1, 0));
  return inc + (wid > 0 ? before : 0u);
}

template <int RAD>
__global__ void __launch_bounds__(kThreads, 1)
k_select_cta(const __grid_constant__ SelCtaArgs a) {
  extern __shared__ __align__(16) float sv[];                // padded votes, kPaddedFloats
  __shared__ __align__(8) int hist[kBins];
  __shared__ unsigned wtot[kWarps];
  __shared__ unsigned sh_prefix;
  __shared__ int sh_need;

  const int tid = threadIdx.x;
  pdl_launch_dependents();
  const int seg = blockIdx.x;
  const int s = seg / a.n_kv_heads, h = seg - s * a.n_kv_heads;
  const int t0 = a.tab.cu_at(s);
  const int len = a.tab.cu_at(s + 1) - t0;
  const int n_hist = max(len - a.window, 0);
  const int n_win = min(len, a.window);
  const int n_seg = a.n_seqs * a.n_kv_heads;
  const long long seg_base = a.tab.hist_at(s) * a.n_kv_heads + (long long)h * n_hist;
  const float* vote = a.vote + seg_base;
  const float pad = a.pool_mode == SLKV_POOL_MAX ? -INFINITY : 0.f;
  pdl_wait();                                // budgets and votes may come from the kernels before this one

  // all of the segment's votes, coalesced, in flight together
  float x[kItems];
#pragma unroll
  for (int k = 0; k < kItems; ++k) {
    const int i = k * kThreads + tid;
    x[k] = i < n_hist ? __ldg(vote + i) : pad;
  }
  const int k_keep = kept_rows(len, a.budgets[h], a.window) - n_win;    // C_H = C - window, clamped

  // packed row where this segment starts = kept rows of all earlier segments (Algorithm 3 l.1-4 per head)
  long long out0;
  {
    unsigned part = 0;                       // < 2^31: the host checks n_kv_heads * total_tokens
    for (int g = tid; g < seg; g += kThreads) {
      const int s2 = g / a.n_kv_heads, h2 = g - s2 * a.n_kv_heads;
      part += (unsigned)kept_rows(a.tab.cu_at(s2 + 1) - a.tab.cu_at(s2), a.budgets[h2], a.window);
    }
    unsigned tot;
    block_incl_scan(part, wtot, &tot);
    out0 = tot;
    if (tid == 0) {
      a.offsets[seg] = (int32_t)tot;
      if (seg == n_seg - 1) {
        const long long all = out0 + k_keep + n_win;
        a.offsets[n_seg] = (int32_t)all;
        if (all > a.capacity && a.status) *a.status = SLKV_ERR_CAPACITY;
      }
    }
  }
  const int src_base = t0 * a.n_kv_heads + h;            // source row of position j: src_base + j * n_kv_heads

  // window rows: always kept, after the history rows
  for (int t = tid; t < n_win; t += kThreads) {
    const long long o = out0 + k_keep + t;
    if (o < a.capacity) {
      a.kept_idx[o] = len - n_win + t;
      a.gather_src[o] = src_base + (len - n_win + t) * a.n_kv_heads;
    }
  }

  const bool need_scores = (k_keep > 0 && k_keep < n_hist) || a.pooled_out != nullptr;
  if (!need_scores) {
    if (k_keep >= n_hist && k_keep > 0) {                              // nothing to drop (Alg. 3 l.1-3)
      for (int i = tid; i < n_hist; i += kThreads)
        if (out0 + i < a.capacity) {
          a.kept_idx[out0 + i] = i;
          a.gather_src[out0 + i] = src_base + i * a.n_kv_heads;
        }
    }
    return;
  }

  // ---- votes to their owners: thread t gets positions [32t - RAD, 32t + 32 + RAD)
#pragma unroll
  for (int k = 0; k < kItems; ++k) sv[padded(k * kThreads + tid)] = x[k];
  if (tid < 32) sv[padded(tid - 32)] = pad;                            // left halo block
  if (tid < 32) sv[padded(kMaxHist + tid)] = pad;                      // right halo block
  __syncthreads();
  const int first = kItems * tid;                                      // first position this thread owns
  const int nv = min(max(n_hist - first, 0), kItems);                  // valid positions among its 32
  unsigned key[kItems];                                                // pooled scores as bit patterns
  {
    float v[kItems + 2 * RAD];
#pragma unroll
    for (int j = 0; j < kItems + 2 * RAD; ++j) v[j] = sv[padded(first - RAD + j)];
    if (a.pool_mode == SLKV_POOL_MAX) {
      // max over [j, j + 2 RAD] by doubling: windows of 2, 4, ... then two overlapping ones
      constexpr int W = 2 * RAD + 1;
      int have = 1;                                                    // v[j] = max of v[j .. j + have - 1]
#pragma unroll
      for (int step = 1; 2 * step <= W; step *= 2) {
#pragma unroll
        for (int j = 0; j + step < kItems + 2 * RAD; ++j) v[j] = fmaxf(v[j], v[j + step]);
        have = 2 * step;
      }
      if (have < W) {
#pragma unroll
        for (int j = 0; j < kItems; ++j) v[j] = fmaxf(v[j], v[j + W - have]);
      }
#pragma unroll
      for (int j = 0; j < kItems; ++j) key[j] = __float_as_uint(v[j]);
    } else {
#pragma unroll
      for (int j = 0; j < kItems; ++j) {
        float acc = v[j];
#pragma unroll
        for (int t = 1; t <= 2 * RAD; ++t) acc += v[j + t];
        key[j] = __float_as_uint(acc / (float)(2 * RAD + 1));
      }
    }
  }
  // the pooled keys also go back to shared memory: later steps visit single positions by index
  __syncthreads();
#pragma unroll
  for (int j = 0; j < kItems; ++j) sv[padded(first + j)] = __uint_as_float(key[j]);
  if (a.pooled_out) {                                                  // coalesced stores from shared memory
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kItems; ++k) {
      const int i = k * kThreads + tid;
      if (i < n_hist) a.pooled_out[seg_base + i] = sv[padded(i)];
    }
  }
  if (k_keep <= 0) return;
  if (k_keep >= n_hist) {                                              // nothing to drop (Alg. 3 l.1-3)
    for (int i = tid; i < n_hist; i += kThreads)
      if (out0 + i < a.capacity) {
        a.kept_idx[out0 + i] = i;
        a.gather_src[out0 + i] = src_base + i * a.n_kv_heads;
      }
    return;
  }

  // ---- k-th largest pooled score: radix descent, one histogram per level
  unsigned prefix = 0;
  int need = k_keep;
  unsigned live = nv >= kItems ? 0xffffffffu : ((1u << nv) - 1u);      // bit j: position first + j still a candidate
#pragma unroll 1
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
    const unsigned dmask = pass == 2 ? 1023u : 2047u;
    reinterpret_cast<int2*>(hist)[tid] = make_int2(0, 0);
    __syncthreads();
    if (pass == 0) {
      // all positions, from registers: one atomic per run of equal digits (max pooling makes neighbours equal)
      unsigned run_digit = key[0] >> 21;
      int run_len = 0;
#pragma unroll
      for (int j = 0; j < kItems; ++j) {
        const unsigned digit = key[j] >> 21;
        if (j < nv) {
          if (digit != run_digit) { atomicAdd(&hist[run_digit], run_len); run_len = 0; run_digit = digit; }
          ++run_len;
        }
      }
      if (run_len > 0) atomicAdd(&hist[run_digit], run_len);
    } else {
      for (unsigned m = live; m != 0; m &= m - 1) {
        const int j = __ffs(m) - 1;
        atomicAdd(&hist[(__float_as_uint(sv[padded(first + j)]) >> shift) & dmask], 1);
      }
    }
    __syncthreads();
    const int2 c = reinterpret_cast<const int2*>(hist)[tid];          // bins 2*tid (c.x) and 2*tid+1 (c.y)
    unsigned tot;
    const unsigned inc = block_incl_scan((unsigned)(c.x + c.y), wtot, &tot);
    const int above_hi = (int)(tot - inc);                             // elements in bins above 2*tid+1
    const int above_lo = above_hi + c.y;                               // above bin 2*tid
    if (above_hi < need && need <= above_hi + c.y) {                   // exactly one bin satisfies this
      sh_prefix = prefix | ((unsigned)(2 * tid + 1) << shift);
      sh_need = need - above_hi;
    } else if (above_lo < need && need <= above_lo + c.x) {
      sh_prefix = prefix | ((unsigned)(2 * tid) << shift);
      sh_need = need - above_lo;
    }
    __syncthreads();
    prefix = sh_prefix;
    need = sh_need;
    if (pass == 0) {
      const unsigned b0 = prefix >> 21;
      unsigned keep = 0;
#pragma unroll
      for (int j = 0; j < kItems; ++j) keep |= ((key[j] >> 21) == b0 ? 1u : 0u) << j;
      live &= keep;
    } else if (pass == 1) {
      const unsigned want = (prefix >> 10) & 2047u;
      unsigned keep = 0;
      for (unsigned m = live; m != 0; m &= m - 1) {
        const int j = __ffs(m) - 1;
        if (((__float_as_uint(sv[padded(first + j)]) >> 10) & 2047u) == want) keep |= 1u << j;
      }
      live = keep;
    }
  }
  const unsigned tau = prefix;            // the k-th largest score; `need` of the positions equal to it are kept

  // ---- ordered compaction: threads own consecutive positions, so thread order is position order
  unsigned gt_mask = 0, eq_mask = 0;
#pragma unroll
  for (int j = 0; j < kItems; ++j) {
    gt_mask |= (key[j] > tau ? 1u : 0u) << j;
    eq_mask |= (key[j] == tau ? 1u : 0u) << j;
  }
  const unsigned valid = nv >= kItems ? 0xffffffffu : ((1u << nv) - 1u);
  gt_mask &= valid; eq_mask &= valid;
  const unsigned my_gt = __popc(gt_mask), my_eq = __popc(eq_mask);
  // both totals are <= 32768: pack them into one scan (equal count in the high half)
  unsigned tot_pack;
  const unsigned inc_pack = block_incl_scan((my_eq << 16) | my_gt, wtot, &tot_pack);
  const int gt_before = (int)((inc_pack & 0xffffu) - my_gt), eq_before = (int)((inc_pack >> 16) - my_eq);
  // of the positions equal to tau, the first `need` (in position order) are kept
  const int eq_take = min(max(need - eq_before, 0), (int)my_eq);
  unsigned eq_kept = 0;
  { unsigned m = eq_mask; for (int t = 0; t < eq_take; ++t) { eq_kept |= m & (0u - m); m &= m - 1; } }
  const unsigned kept_mask = gt_mask | eq_kept;
  // a kept position's output row: kept ones before it = (greater before) + min(equal before, need)
  long long o = out0 + gt_before + min(eq_before, need);
  for (unsigned m = kept_mask; m != 0; m &= m - 1, ++o) {
    const int j = __ffs(m) - 1;
    if (o < a.capacity) {
      a.kept_idx[o] = first + j;
      a.gather_src[o] = src_base + (first + j) * a.n_kv_heads;
    }
  }
}

}  // namespace

bool select_cta_supported(const Problem& pb) {
  return pb.max_hist <= kMaxHist && (pb.p.pool_kernel >> 1) <= kMaxRadius;
}

cudaError_t launch_select_cta(const Problem& pb, float* pooled_out, const int32_t* budgets, int32_t* offsets,
                              int32_t* kept_idx, int64_t capacity, int32_t* status, cudaStream_t st, int* launches) {
  typedef void (*Kern)(const SelCtaArgs);
  static const Kern kerns[kMaxRadius + 1] = {k_select_cta<0>, k_select_cta<1>, k_select_cta<2>, k_select_cta<3>,
                                             k_select_cta<4>};
  const size_t smem = (size_t)kPaddedFloats * sizeof(float);
  static thread_local int configured_dev = -1;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (configured_dev != dev) {
    for (int r = 0; r <= kMaxRadius; ++r) {
      e = cudaFuncSetAttribute(kerns[r], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    configured_dev = dev;
  }
  SelCtaArgs a;
  a.vote = pb.vote; a.pooled_out = pooled_out; a.budgets = budgets; a.offsets = offsets; a.kept_idx = kept_idx;
  a.gather_src = pb.gather_src; a.status = status;
  a.n_seqs = pb.p.n_seqs; a.n_kv_heads = pb.p.n_kv_heads; a.window = pb.p.window; a.pool_mode = pb.p.pool_mode;
  a.capacity = capacity; a.tab = pb.tab;
  LaunchScope scope(KID_SELECT, st, launches);
  return launch_pdl(kerns[pb.p.pool_kernel >> 1], dim3((unsigned)pb.n_seg), dim3(kThreads), smem, st, 1, a);
}

}  // namespace slkv
