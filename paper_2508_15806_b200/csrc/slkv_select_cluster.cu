// Pooling + per-head variable-k selection, one thread-block cluster per (sequence, KV head) segment
// (Sec. 3.4, Eq. 8; Algorithm 3 lines 1-4, 7-8).
//
// The segment's votes are split evenly over the cluster's CTAs and stay in shared memory from the first
// read to the last: pooled in place, then searched for the k-th largest value by a 4 x 8-bit radix
// descent whose 256-bin histograms are summed across the cluster through distributed shared memory, then
// compacted in position order.  Integer counters only, so the result does not depend on timing.
#include <cooperative_groups.h>

#include "slkv_internal.cuh"

namespace cg = cooperative_groups;

namespace slkv {
namespace {

constexpr int kThreads = 1024;
constexpr int kMaxItems = 16;                         // slice elements per thread kept in shared memory
constexpr int kMaxSlice = kThreads * kMaxItems;       // 16384 scores per CTA
constexpr int kMaxCluster = 8;

struct SelArgs {
  const float* vote;
  float* pooled_out;          // optional
  SeqTables tab;
  const int32_t* budgets;
  int32_t* offsets;
  int32_t* kept_idx;
  int32_t* status;
  int n_seqs, n_kv_heads, window, pool_kernel, pool_mode;
  int keys_off;               // float index in shared memory where the pooled keys start
  long long capacity;
};

__device__ __forceinline__ int kept_rows(int len, int budget, int window) { return min(len, max(budget, window)); }

template <typename T>
__device__ __forceinline__ T block_excl_scan(T v, T* warp_tot /*[32]*/, T* total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  T inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    T n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  __syncthreads();
  if (lane == 31) warp_tot[wid] = inc;
  __syncthreads();
  T base = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) {
    T t = warp_tot[w];
    if (w < wid) base += t;
    tot += t;
  }
  *total = tot;
  return base + inc - v;
}

__global__ void __launch_bounds__(kThreads, 1)
k_select_cluster(const __grid_constant__ SelArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ int hist[2][256];
  __shared__ long long wt[32];
  __shared__ int cta_tot[2];                 // this CTA's (greater, equal) counts, read by the others
  __shared__ unsigned sh_prefix;
  __shared__ int sh_need;
  __shared__ long long sh_out0;

  cg::cluster_group cluster = cg::this_cluster();
  const int CS = (int)cluster.num_blocks();
  const int rank = (int)cluster.block_rank();
  const int tid = threadIdx.x, lane = tid & 31;
  pdl_launch_dependents();
  pdl_wait();
  const int seg = blockIdx.x / CS;
  const int s = seg / a.n_kv_heads, h = seg - s * a.n_kv_heads;
  const int len = a.tab.cu_at(s + 1) - a.tab.cu_at(s);
  const int n_hist = max(len - a.window, 0);
  const int n_win = min(len, a.window);
  const int k_keep = kept_rows(len, a.budgets[h], a.window) - n_win;    // C_H = C - window, clamped
  const int n_seg = a.n_seqs * a.n_kv_heads;

  // packed row where this segment starts = kept rows of all earlier segments (Algorithm 3 l.1-4 per head)
  {
    long long part = 0;
    for (int g = tid; g < seg; g += kThreads) {
      const int s2 = g / a.n_kv_heads, h2 = g - s2 * a.n_kv_heads;
      part += kept_rows(a.tab.cu_at(s2 + 1) - a.tab.cu_at(s2), a.budgets[h2], a.window);
    }
    long long tot;
    block_excl_scan<long long>(part, wt, &tot);
    if (tid == 0) {
      sh_out0 = tot;
      if (rank == 0) {
        a.offsets[seg] = (int32_t)tot;
        if (seg == n_seg - 1) {
          const long long all = tot + k_keep + n_win;
          a.offsets[n_seg] = (int32_t)all;
          if (all > a.capacity && a.status) *a.status = SLKV_ERR_CAPACITY;
        }
      }
    }
    __syncthreads();
  }
  const long long out0 = sh_out0;

  // this CTA's slice [lo, hi) of the history
  const int per = ((n_hist + CS - 1) / CS + 3) & ~3;
  const int lo = min(rank * per, n_hist), hi = min(lo + per, n_hist);
  const int n_own = hi - lo;
  const long long seg_base = a.tab.hist_at(s) * a.n_kv_heads + (long long)h * n_hist;
  const float* vote = a.vote + seg_base;
  const int r = a.pool_kernel >> 1;
  float* sv = reinterpret_cast<float*>(smem_raw);                    // votes of [lo - r, hi + r), then pooled keys
  unsigned* keys = reinterpret_cast<unsigned*>(smem_raw) + a.keys_off;          // pooled bit patterns of [lo, hi)

  // window rows: always kept, after the history rows
  if (rank == 0)
    for (int t = tid; t < n_win; t += kThreads) {
      const long long o = out0 + k_keep + t;
      if (o < a.capacity) a.kept_idx[o] = len - n_win + t;
    }

  const bool need_scores = (k_keep > 0 && k_keep < n_hist) || a.pooled_out != nullptr;
  if (need_scores) {
    for (int i = tid; i < n_own + 2 * r; i += kThreads) {
      const int j = lo - r + i;
      sv[i] = (j >= 0 && j < n_hist) ? vote[j] : (a.pool_mode == SLKV_POOL_MAX ? -INFINITY : 0.f);
    }
    __syncthreads();
    for (int i = tid; i < n_own; i += kThreads) {
      float acc;
      if (a.pool_mode == SLKV_POOL_MAX) {
        acc = sv[i];
        for (int t = 1; t <= 2 * r; ++t) acc = fmaxf(acc, sv[i + t]);
      } else {
        acc = 0.f;
        for (int t = 0; t <= 2 * r; ++t) acc += sv[i + t];
        acc = acc / (float)a.pool_kernel;
      }
      keys[i] = __float_as_uint(acc);
      if (a.pooled_out) a.pooled_out[seg_base + lo + i] = acc;
    }
    __syncthreads();
  }

  if (k_keep <= 0) return;                                           // uniform over the cluster
  if (k_keep >= n_hist) {                                            // nothing to drop (Alg. 3 l.1-3)
    for (int i = tid; i < n_own; i += kThreads)
      if (out0 + lo + i < a.capacity) a.kept_idx[out0 + lo + i] = lo + i;
    return;
  }

  // ---- k-th largest pooled score of the segment: radix descent, histograms summed over the cluster
  unsigned prefix = 0, mask = 0;
  int need = k_keep;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    int* hl = hist[pass & 1];
    if (tid < 256) hl[tid] = 0;
    __syncthreads();
    for (int i0 = 0; i0 < n_own; i0 += kThreads) {
      const int i = i0 + tid;
      const bool in = i < n_own;
      const unsigned v = in ? keys[i] : 0u;
      const bool live = in && ((v & mask) == prefix);
      const unsigned digit = (v >> shift) & 255u;
      // one shared-memory atomic per distinct digit in the warp
      const unsigned act = __ballot_sync(0xffffffffu, live);
      if (live) {
        const unsigned peers = __match_any_sync(act, digit);
        if (lane == __ffs(peers) - 1) atomicAdd(&hl[digit], __popc(peers));
      }
    }
    cluster.sync();                                                  // every CTA's histogram is complete
    int tot = 0;
    if (tid < 256)
      for (int c = 0; c < CS; ++c) tot += cluster.map_shared_rank(hl, c)[tid];
    // suffix sums over the 256 bins (bin 255 first): the digit where the count from the top reaches `need`
    const int rev = (tid < 256) ? tot : 0;
    // thread t holds bin t; scan in reversed bin order = inclusive suffix sum
    int inc = rev;
    {
      // suffix scan via prefix scan on reversed index: use shuffles + warp totals (8 warps matter)
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_down_sync(0xffffffffu, inc, o);
        if (lane + o < 32) inc += n;
      }
      __shared__ int wsum[8];
      if (tid < 256 && lane == 0) wsum[tid >> 5] = inc;
      __syncthreads();
      if (tid < 256) {
        for (int w = (tid >> 5) + 1; w < 8; ++w) inc += wsum[w];
        const int above = inc - rev;                                 // elements in higher bins
        if (above < need && need <= inc) {                           // exactly one bin satisfies this
          sh_prefix = prefix | ((unsigned)tid << shift);
          sh_need = need - above;
        }
      }
      __syncthreads();
    }
    prefix = sh_prefix;
    need = sh_need;
    mask |= 255u << shift;
  }
  const unsigned tau = prefix;            // the k-th largest score; `need` of the positions equal to it are kept

  // ---- ordered compaction: thread t owns the contiguous run [t*items, (t+1)*items) of the slice
  const int items = (n_own + kThreads - 1) / kThreads;
  int my_gt = 0, my_eq = 0;
  for (int e = 0; e < items; ++e) {
    const int i = tid * items + e;
    if (i < n_own) {
      const unsigned v = keys[i];
      my_gt += v > tau;
      my_eq += v == tau;
    }
  }
  long long tot_pack;
  const long long ex_pack = block_excl_scan<long long>(((long long)my_eq << 32) | (unsigned)my_gt, wt, &tot_pack);
  if (tid == 0) { cta_tot[0] = (int)(tot_pack & 0xffffffffll); cta_tot[1] = (int)(tot_pack >> 32); }
  cluster.sync();
  int gt_before = (int)(ex_pack & 0xffffffffll), eq_before = (int)(ex_pack >> 32);
  for (int c = 0; c < rank; ++c) {
    const int* ct = cluster.map_shared_rank(cta_tot, c);
    gt_before += ct[0];
    eq_before += ct[1];
  }
  for (int e = 0; e < items; ++e) {
    const int i = tid * items + e;
    if (i < n_own) {
      const unsigned v = keys[i];
      const bool gt = v > tau, eq = v == tau;
      if (gt || (eq && eq_before < need)) {
        const long long o = out0 + gt_before + min(eq_before, need);
        if (o < a.capacity) a.kept_idx[o] = lo + i;
      }
      gt_before += gt;
      eq_before += eq;
    }
  }
  cluster.sync();                          // nobody leaves while its shared memory may still be read
}

}  // namespace

int select_cluster_size(const Problem& pb) {
  // enough CTAs per segment to keep every slice in shared memory, and to spread few segments over the SMs
  int cs = 1;
  while (cs < kMaxCluster && (cs * pb.n_seg * 2 <= 148 || (pb.max_hist + cs - 1) / cs + 4 > kMaxSlice)) cs *= 2;
  return cs;
}

bool select_cluster_supported(const Problem& pb) {
  const int cs = select_cluster_size(pb);
  return (pb.max_hist + cs - 1) / cs + 4 <= kMaxSlice && pb.p.pool_kernel <= 129;
}

cudaError_t launch_select_cluster(const Problem& pb, float* pooled_out, const int32_t* budgets, int32_t* offsets,
                                  int32_t* kept_idx, int64_t capacity, int32_t* status, cudaStream_t st,
                                  int* launches) {
  const int cs = select_cluster_size(pb);
  const int per = (((pb.max_hist + cs - 1) / cs + 3) & ~3);
  const int keys_off = (per + 2 * (pb.p.pool_kernel >> 1) + 3) & ~3;
  const size_t smem = (size_t)(keys_off + per) * sizeof(float);
  static thread_local int configured_dev = -1;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (configured_dev != dev) {
    e = cudaFuncSetAttribute(k_select_cluster, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
    if (e != cudaSuccess) return e;
    configured_dev = dev;
  }
  SelArgs a;
  a.vote = pb.vote; a.pooled_out = pooled_out; a.tab = pb.tab; a.budgets = budgets;
  a.offsets = offsets; a.kept_idx = kept_idx; a.status = status;
  a.n_seqs = pb.p.n_seqs; a.n_kv_heads = pb.p.n_kv_heads; a.window = pb.p.window;
  a.pool_kernel = pb.p.pool_kernel; a.pool_mode = pb.p.pool_mode; a.capacity = capacity;
  a.keys_off = keys_off;

  LaunchScope scope(KID_SELECT, st, launches);
  return launch_pdl(k_select_cluster, dim3((unsigned)(pb.n_seg * cs)), dim3(kThreads), smem, st, cs, a);
}

}  // namespace slkv
