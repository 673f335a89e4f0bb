// Stage-2 KV budget allocation (Sec. 3.3, Eq. 6; Algorithm 2), one CTA, fp64 in a fixed operation order.
//
// Head (i, j) gets  fixed + share_ij  where the shares split the dynamic pool D = total - N*fixed in
// proportion to Algorithm 2's weight (0.01 + L_i/L_s) * (inf_ij/L_s) and are rounded by largest
// remainder so that they sum to D exactly.  Options: the head share over the layer's own sum (the prose under
// Eq. 6), a per-head cap whose excess is handed on to the other heads, Algorithm 2's own rounding.
// The sums over heads and layers run sequentially in index order on one thread and every product / quotient
// is a separately rounded IEEE operation (__dadd_rn / __dmul_rn / __ddiv_rn stop the compiler from fusing
// them), so the integers that come out do not depend on the launch shape.
#include "slkv_internal.cuh"

namespace slkv {
namespace {

constexpr int kAllocThreads = 1024;

struct AllocOpts {
  int within_layer;      // head share over the layer's sum (prose under Eq. 6) instead of the grand sum (Algorithm 2)
  int paper_rounding;    // Algorithm 2's own last line instead of the normalisation
  long long cap;         // < 0: none
};

// Algorithm 2's weight of head a = (layer i, head j): (0.01 + L_i / L_s) * S_ij; 1 for every head when no head has
// any influence.
__device__ __forceinline__ double head_weight(const float* inf, const double* La, double Ls, int H, int a,
                                              bool uniform, bool within_layer) {
  if (uniform) return 1.0;
  const int i = a / H;
  const double lw = __dadd_rn(kLayerFloor, __ddiv_rn(La[i], Ls));      // 0.01 + L_{i,h}
  double share;
  if (within_layer) share = La[i] > 0.0 ? __ddiv_rn((double)inf[a], La[i]) : __ddiv_rn(1.0, (double)H);
  else share = __ddiv_rn((double)inf[a], Ls);                          // S_{j,h}
  return __dmul_rn(lw, share);
}

__device__ long long block_sum_ll(long long v, long long* red) {
  __syncthreads();
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  long long t = 0;
  for (int w = 0; w < kAllocThreads / 32; ++w) t += red[w];
  return t;
}

__global__ void __launch_bounds__(kAllocThreads, 1)
k_alloc(const float* __restrict__ inf, int L, int H, int fixed, long long total, const AllocOpts opt,
        int32_t* __restrict__ budgets, int32_t* __restrict__ status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int N = L * H;
  double* rem = reinterpret_cast<double*>(smem_raw);       // [N] fractional parts
  double* La = rem + N;                                    // [L] layer sums
  unsigned char* active = reinterpret_cast<unsigned char*>(La + L);   // [N] head still below the cap
  __shared__ long long red[kAllocThreads / 32];
  __shared__ double sh_Ls, sh_W;
  __shared__ int sh_bad, sh_uniform, sh_flat, sh_n_active;
  const int tid = threadIdx.x;
  const long long D = total - (long long)N * fixed;
  const bool within = opt.within_layer != 0;
  pdl_launch_dependents();
  pdl_wait();

  if (tid == 0) sh_bad = 0;
  __syncthreads();
  for (int a = tid; a < N; a += kAllocThreads) {
    float x = inf[a];
    if (!(x >= 0.0f) || !(x <= 3.402823466e38f)) sh_bad = 1;         // negative, NaN or infinite
  }
  __syncthreads();
  if (sh_bad) {
    if (tid == 0 && status) *status = SLKV_ERR_NEG_INF_SC;
    return;
  }

  // layer sums: one thread per layer, each sequential over its heads (index order)
  for (int i = tid; i < L; i += kAllocThreads) {
    double acc = 0.0;
    for (int j = 0; j < H; ++j) acc = __dadd_rn(acc, (double)inf[i * H + j]);
    La[i] = acc;
  }
  __syncthreads();
  if (tid == 0) {
    double Ls = 0.0;
    for (int i = 0; i < L; ++i) Ls = __dadd_rn(Ls, La[i]);
    sh_Ls = Ls;
    sh_uniform = !(Ls > 0.0);
  }
  __syncthreads();
  const double Ls = sh_Ls;
  const bool uniform = sh_uniform != 0;

  if (opt.paper_rounding) {
    // Algorithm 2's own last line: C = floor(max(0, fixed + D * w) + 0.5), clipped at the cap; nothing is normalised
    for (int a = tid; a < N; a += kAllocThreads) {
      const double w = uniform ? __ddiv_rn(1.0, (double)N) : head_weight(inf, La, Ls, H, a, false, within);
      const double b = __dadd_rn((double)fixed, __dmul_rn((double)D, w));
      long long c = (long long)floor(__dadd_rn(fmax(0.0, b), 0.5));
      if (opt.cap >= 0 && c > opt.cap) c = opt.cap;
      budgets[a] = (int32_t)c;
    }
    return;
  }

  // Heads that would rise above the cap are filled and taken out, the rest share what is left, until none does
  // (without a cap: one round, nobody is taken out).  The sum of the weights runs sequentially in index order.
  for (int a = tid; a < N; a += kAllocThreads) active[a] = 1;
  const long long room = opt.cap >= 0 ? opt.cap - fixed : -1;
  long long d_rem = D;
  while (true) {
    __syncthreads();
    if (tid == 0) {
      double W = 0.0;
      int n_active = 0;
      for (int a = 0; a < N; ++a)
        if (active[a]) { W = __dadd_rn(W, head_weight(inf, La, Ls, H, a, uniform, within)); ++n_active; }
      const int flat = !(W > 0.0);                                    // every weight left underflowed: share evenly
      if (flat) W = (double)n_active;
      sh_W = W; sh_flat = flat; sh_n_active = n_active;
    }
    __syncthreads();
    if (room < 0 || sh_n_active == 0) break;
    const double W = sh_W;
    const bool flat = sh_flat != 0;
    long long filled = 0;
    for (int a = tid; a < N; a += kAllocThreads) {
      if (!active[a]) continue;
      const double wgt = flat ? 1.0 : head_weight(inf, La, Ls, H, a, uniform, within);
      const double q = __ddiv_rn(__dmul_rn((double)d_rem, wgt), W);
      if (q >= (double)room) { active[a] = 0; budgets[a] = (int32_t)room; ++filled; }
    }
    filled = block_sum_ll(filled, red);
    if (filled == 0) break;
    d_rem -= filled * room;
  }
  const double W = sh_W;
  const bool flat = sh_flat != 0;
  const int n_active = sh_n_active;

  // quotas, floors, remainders of the heads still below the cap
  long long fsum = 0;
  for (int a = tid; a < N; a += kAllocThreads) {
    if (!active[a]) continue;
    const double wgt = flat ? 1.0 : head_weight(inf, La, Ls, H, a, uniform, within);
    const double q = __ddiv_rn(__dmul_rn((double)d_rem, wgt), W);
    const double fl = floor(q);
    rem[a] = __dadd_rn(q, -fl);
    const long long f = (long long)fl;
    budgets[a] = (int32_t)f;                                          // floors for now
    fsum += f;
  }
  long long Rleft = d_rem - block_sum_ll(fsum, red);
  if (n_active > 0 && Rleft >= n_active) {                            // not reachable in exact arithmetic
    const long long each = Rleft / n_active;
    for (int a = tid; a < N; a += kAllocThreads)
      if (active[a]) budgets[a] += (int32_t)each;
    Rleft -= each * n_active;
  }
  __syncthreads();
  if (Rleft > 0) {
    // largest remainder first, ties -> lower index: head a gets +1 iff fewer than Rleft heads precede it
    for (int a = tid; a < N; a += kAllocThreads) {
      if (!active[a]) continue;
      const double ra = rem[a];
      int rank = 0;
      for (int b = 0; b < N; ++b) {
        if (!active[b]) continue;
        const double rb = rem[b];
        rank += (rb > ra) || (rb == ra && b < a);
      }
      if (rank < Rleft) budgets[a] += 1;
    }
  }
  while (Rleft < 0) {
    // floors overshot the pool (rounding): take one back from the smallest remainders, ties -> higher index
    __syncthreads();
    long long taken = 0;
    int dec[(16384 + kAllocThreads - 1) / kAllocThreads];
    int nd = 0;
    for (int a = tid; a < N; a += kAllocThreads, ++nd) {
      dec[nd] = 0;
      if (!active[a] || budgets[a] <= 0) continue;
      const double ra = rem[a];
      int rank = 0;
      for (int b = 0; b < N; ++b) {
        if (!active[b] || budgets[b] <= 0) continue;
        const double rb = rem[b];
        rank += (rb < ra) || (rb == ra && b > a);
      }
      if (rank < -Rleft) { dec[nd] = 1; ++taken; }
    }
    __syncthreads();
    nd = 0;
    for (int a = tid; a < N; a += kAllocThreads, ++nd)
      if (dec[nd]) budgets[a] -= 1;
    Rleft += block_sum_ll(taken, red);
  }
  __syncthreads();
  for (int a = tid; a < N; a += kAllocThreads) budgets[a] += fixed;
}

}  // namespace

cudaError_t launch_alloc(const float* inf, int n_layers, int n_heads, int fixed, long long total, int within_layer,
                         int paper_rounding, long long cap, int32_t* budgets, int32_t* status, cudaStream_t st) {
  const size_t n = (size_t)n_layers * n_heads;
  size_t smem = (n + n_layers) * sizeof(double) + n;
  static thread_local int configured_dev = -1;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (configured_dev != dev) {
    e = cudaFuncSetAttribute(k_alloc, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    configured_dev = dev;
  }
  AllocOpts opt;
  opt.within_layer = within_layer; opt.paper_rounding = paper_rounding; opt.cap = cap;
  int launches = 0;
  LaunchScope scope(KID_ALLOC, st, &launches);
  k_alloc<<<1, kAllocThreads, smem, st>>>(inf, n_layers, n_heads, fixed, total, opt, budgets, status);
  return cudaGetLastError();
}

}  // namespace slkv
