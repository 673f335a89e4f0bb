// Pooling + per-head variable-k selection, one thread-block cluster per (sequence, KV head) segment
// (Sec. 3.4, Eq. 8; Algorithm 3 lines 1-4, 7-8).
//
// The segment's votes are split evenly over the cluster's CTAs and stay in shared memory from the first
// read to the last: pooled in place, then searched for the k-th largest value by a radix descent over the
// float bit patterns (11 + 11 + 10 bits; scores are >= 0, so unsigned order = float order) whose
// histograms are summed across the cluster through distributed shared memory, then compacted in position
// order.  Integer counters only, so the result does not depend on timing.
#include <cooperative_groups.h>

#include "slkv_internal.cuh"

namespace cg = cooperative_groups;

namespace slkv {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxItems = 16;                         // slice elements per thread kept in shared memory
constexpr int kMaxSlice = kThreads * kMaxItems;       // 16384 scores per CTA
constexpr int kMaxCluster = 8;
constexpr int kBins = 2048;

struct SelArgs {
  const float* vote;
  float* pooled_out;          // optional
  SeqTables tab;
  const int32_t* budgets;
  int32_t* offsets;
  int32_t* kept_idx;
  int32_t* gather_src;        // per packed row: token * n_kv_heads + head of the source row
  int32_t* status;
  int n_seqs, n_kv_heads, window, pool_kernel, pool_mode;
  int keys_off;               // float index in shared memory where the pooled keys start
  long long capacity;
};

__device__ __forceinline__ int kept_rows(int len, int budget, int window) { return min(len, max(budget, window)); }

// Inclusive scan of one int per thread over the CTA in thread order; *total = CTA sum.  `wtot` is 32 ints.
__device__ __forceinline__ int block_incl_scan(int v, int* wtot, int* total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  __syncthreads();                       // wtot may still be read from an earlier call
  if (lane == 31) wtot[wid] = inc;
  __syncthreads();
  int w = wtot[lane];                    // every warp scans the 32 warp totals itself
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, w, o);
    if (lane >= o) w += n;
  }
  *total = __shfl_sync(0xffffffffu, w, 31);
  const int before = __shfl_sync(0xffffffffu, w, max(wid - 1, 0));
  return inc + (wid > 0 ? before : 0);
}

__global__ void __launch_bounds__(kThreads, 1)
k_select_cluster(const __grid_constant__ SelArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ __align__(8) int hist[kBins];
  __shared__ __align__(16) unsigned short hist16[2][kBins];   // a slice holds <= 16384 scores: counts fit 16 bits
  __shared__ int wtot[kWarps];
  __shared__ __align__(8) int cta_tot[2];    // this CTA's (greater, equal) counts, read by the others
  __shared__ int before_sh[2];
  __shared__ unsigned sh_prefix;
  __shared__ int sh_need;

  cg::cluster_group cluster = cg::this_cluster();
  const int CS = (int)cluster.num_blocks();
  const int rank = (int)cluster.block_rank();
  const int tid = threadIdx.x, lane = tid & 31;
  pdl_launch_dependents();
  const int seg = blockIdx.x / CS;
  const int s = seg / a.n_kv_heads, h = seg - s * a.n_kv_heads;
  const int t0 = a.tab.cu_at(s);
  const int len = a.tab.cu_at(s + 1) - t0;
  const int n_hist = max(len - a.window, 0);
  const int n_win = min(len, a.window);
  const int n_seg = a.n_seqs * a.n_kv_heads;
  // this CTA's slice [lo, hi) of the history
  const int per = ((n_hist + CS - 1) / CS + 3) & ~3;
  const int lo = min(rank * per, n_hist), hi = min(lo + per, n_hist);
  const int n_own = hi - lo;
  const long long seg_base = a.tab.hist_at(s) * a.n_kv_heads + (long long)h * n_hist;
  const float* vote = a.vote + seg_base;
  const int r = a.pool_kernel >> 1;
  float* sv = reinterpret_cast<float*>(smem_raw);                    // votes of [lo - r, hi + r)
  unsigned* keys = reinterpret_cast<unsigned*>(smem_raw) + a.keys_off;          // pooled bit patterns of [lo, hi)
  const float pad = a.pool_mode == SLKV_POOL_MAX ? -INFINITY : 0.f;
  pdl_wait();                                // budgets and votes may come from the kernels before this one
  // The first 8192 votes of the slice start their way from L2 now, under the offset arithmetic below.
  float x0[8];
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const int i = u * kThreads + tid, j = lo - r + i;
    x0[u] = (i < n_own + 2 * r && j >= 0 && j < n_hist) ? __ldg(vote + j) : pad;
  }
  const int k_keep = kept_rows(len, a.budgets[h], a.window) - n_win;    // C_H = C - window, clamped

  // packed row where this segment starts = kept rows of all earlier segments (Algorithm 3 l.1-4 per head)
  long long out0;
  {
    int part = 0;                            // < 2^31: the host checks n_kv_heads * total_tokens
    for (int g = tid; g < seg; g += kThreads) {
      const int s2 = g / a.n_kv_heads, h2 = g - s2 * a.n_kv_heads;
      part += kept_rows(a.tab.cu_at(s2 + 1) - a.tab.cu_at(s2), a.budgets[h2], a.window);
    }
    int tot;
    block_incl_scan(part, wtot, &tot);
    out0 = tot;
    if (tid == 0 && rank == 0) {
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
  if (rank == 0)
    for (int t = tid; t < n_win; t += kThreads) {
      const long long o = out0 + k_keep + t;
      if (o < a.capacity) {
        a.kept_idx[o] = len - n_win + t;
        a.gather_src[o] = src_base + (len - n_win + t) * a.n_kv_heads;
      }
    }

  const bool need_scores = (k_keep > 0 && k_keep < n_hist) || a.pooled_out != nullptr;
  if (need_scores) {
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = u * kThreads + tid;
      if (i < n_own + 2 * r) sv[i] = x0[u];
    }
    for (int i0 = 8 * kThreads; i0 < n_own + 2 * r; i0 += 8 * kThreads) {        // eight loads in flight per thread
      float x[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = i0 + u * kThreads + tid, j = lo - r + i;
        x[u] = (i < n_own + 2 * r && j >= 0 && j < n_hist) ? __ldg(vote + j) : pad;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = i0 + u * kThreads + tid;
        if (i < n_own + 2 * r) sv[i] = x[u];
      }
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
      if (out0 + lo + i < a.capacity) {
        a.kept_idx[out0 + lo + i] = lo + i;
        a.gather_src[out0 + lo + i] = src_base + (lo + i) * a.n_kv_heads;
      }
    return;
  }

  // ---- k-th largest pooled score of the segment: radix descent, histograms summed over the cluster
  unsigned prefix = 0, mask = 0;
  int need = k_keep;
#pragma unroll 1
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
    const unsigned dmask = pass == 2 ? 1023u : 2047u;
    reinterpret_cast<int2*>(hist)[tid] = make_int2(0, 0);
    __syncthreads();
    for (int i0 = 0; i0 < n_own; i0 += kThreads) {
      const int i = i0 + tid;
      const bool in = i < n_own;
      const unsigned v = in ? keys[i] : 0u;
      const bool live = in && ((v & mask) == prefix);
      const unsigned digit = (v >> shift) & dmask;
      // one shared-memory atomic per distinct digit in the warp
      const unsigned act = __ballot_sync(0xffffffffu, live);
      if (live) {
        const unsigned peers = __match_any_sync(act, digit);
        if (lane == __ffs(peers) - 1) atomicAdd(&hist[digit], __popc(peers));
      }
    }
    __syncthreads();
    unsigned* h16 = reinterpret_cast<unsigned*>(hist16[pass & 1]);   // two passes apart: nobody still reads it
    {
      const int2 mine = reinterpret_cast<const int2*>(hist)[tid];
      h16[tid] = (unsigned)mine.x | ((unsigned)mine.y << 16);
    }
    cluster.sync();                                                  // every CTA's histogram is complete
    // Threads 0..255 sum bins 8t .. 8t+7 over the cluster: one 16-byte remote read per CTA and thread, all
    // in flight together.
    int cnt[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (tid < kBins / 8) {
      uint4 part[kMaxCluster];
#pragma unroll
      for (int c = 0; c < kMaxCluster; ++c)
        part[c] = c < CS ? reinterpret_cast<const uint4*>(cluster.map_shared_rank(h16, c))[tid] : make_uint4(0, 0, 0, 0);
#pragma unroll
      for (int c = 0; c < kMaxCluster; ++c) {
        cnt[0] += (int)(part[c].x & 0xffffu); cnt[1] += (int)(part[c].x >> 16);
        cnt[2] += (int)(part[c].y & 0xffffu); cnt[3] += (int)(part[c].y >> 16);
        cnt[4] += (int)(part[c].z & 0xffffu); cnt[5] += (int)(part[c].z >> 16);
        cnt[6] += (int)(part[c].w & 0xffffu); cnt[7] += (int)(part[c].w >> 16);
      }
    }
    int mine = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) mine += cnt[e];
    int tot;
    const int inc = block_incl_scan(mine, wtot, &tot);
    int above = tot - inc;                                           // elements in bins above 8*tid+7
    if (above < need && need <= above + mine) {                      // the bin lies in this thread's eight
#pragma unroll
      for (int e = 7; e >= 0; --e) {
        if (above < need && need <= above + cnt[e]) {
          sh_prefix = prefix | ((unsigned)(8 * tid + e) << shift);
          sh_need = need - above;
        }
        above += cnt[e];
      }
    }
    __syncthreads();
    prefix = sh_prefix;
    need = sh_need;
    mask |= dmask << shift;
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
  // both counts are <= 16384: pack them into one scan
  int tot_pack;
  const int inc_pack = block_incl_scan((my_eq << 16) | my_gt, wtot, &tot_pack);
  if (tid == 0) { cta_tot[0] = tot_pack & 0xffff; cta_tot[1] = tot_pack >> 16; }
  cluster.sync();
  if (tid < 32) {                          // (greater, equal) counts of the CTAs before this one
    int2 ct = make_int2(0, 0);
    if (lane < rank) ct = *reinterpret_cast<const int2*>(cluster.map_shared_rank(cta_tot, lane));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      ct.x += __shfl_xor_sync(0xffffffffu, ct.x, o);
      ct.y += __shfl_xor_sync(0xffffffffu, ct.y, o);
    }
    if (lane == 0) { before_sh[0] = ct.x; before_sh[1] = ct.y; }
  }
  __syncthreads();
  int gt_before = (inc_pack & 0xffff) - my_gt + before_sh[0], eq_before = (inc_pack >> 16) - my_eq + before_sh[1];
  for (int e = 0; e < items; ++e) {
    const int i = tid * items + e;
    if (i < n_own) {
      const unsigned v = keys[i];
      const bool gt = v > tau, eq = v == tau;
      if (gt || (eq && eq_before < need)) {
        const long long o = out0 + gt_before + min(eq_before, need);
        if (o < a.capacity) {
          a.kept_idx[o] = lo + i;
          a.gather_src[o] = src_base + (lo + i) * a.n_kv_heads;
        }
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
  a.offsets = offsets; a.kept_idx = kept_idx; a.gather_src = pb.gather_src; a.status = status;
  a.n_seqs = pb.p.n_seqs; a.n_kv_heads = pb.p.n_kv_heads; a.window = pb.p.window;
  a.pool_kernel = pb.p.pool_kernel; a.pool_mode = pb.p.pool_mode; a.capacity = capacity;
  a.keys_off = keys_off;

  LaunchScope scope(KID_SELECT, st, launches);
  return launch_pdl(k_select_cluster, dim3((unsigned)(pb.n_seg * cs)), dim3(kThreads), smem, st, cs, a);
}

}  // namespace slkv
