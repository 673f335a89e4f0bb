// Stage-2 KV budget allocation (Sec. 3.3, Eq. 6; Algorithm 2), one CTA, fp64 in a fixed operation order.
//
// Head (i, j) gets  fixed + share_ij  where the shares split the dynamic pool D = total - N*fixed in
// proportion to Algorithm 2's weight (0.01 + L_i/L_s) * (inf_ij/L_s) and are rounded by largest
// remainder so that they sum to D exactly.  The sums over heads and layers run sequentially in index
// order on one thread and every product / quotient is a separately rounded IEEE operation
// (__dadd_rn / __dmul_rn / __ddiv_rn stop the compiler from fusing them), so the integers that come out
// do not depend on the launch shape.
#include "slkv_internal.cuh"

namespace slkv {
namespace {

constexpr int kAllocThreads = 1024;

__device__ __forceinline__ double head_weight(const float* inf, const double* La, double Ls, int H, int a,
                                              bool uniform) {
  if (uniform) return 1.0;
  int i = a / H;
  double lw = __dadd_rn(kLayerFloor, __ddiv_rn(La[i], Ls));            // 0.01 + L_{i,h}
  return __dmul_rn(lw, __ddiv_rn((double)inf[a], Ls));                 // * S_{j,h}
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
k_alloc(const float* __restrict__ inf, int L, int H, int fixed, long long total, int32_t* __restrict__ budgets,
        int32_t* __restrict__ status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int N = L * H;
  double* rem = reinterpret_cast<double*>(smem_raw);       // [N] fractional parts
  double* La = rem + N;                                    // [L] layer sums
  __shared__ long long red[kAllocThreads / 32];
  __shared__ double sh_Ls, sh_W;
  __shared__ int sh_bad, sh_uniform;
  const int tid = threadIdx.x;
  const long long D = total - (long long)N * fixed;
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
    int uniform = !(Ls > 0.0);
    double W = 0.0;
    if (!uniform) {
      for (int a = 0; a < N; ++a) W = __dadd_rn(W, head_weight(inf, La, Ls, H, a, false));
      if (!(W > 0.0)) uniform = 1;
    }
    if (uniform) W = (double)N;
    sh_W = W;
    sh_uniform = uniform;
  }
  __syncthreads();
  const double Ls = sh_Ls, W = sh_W;
  const bool uniform = sh_uniform != 0;

  // quotas, floors, remainders
  long long fsum = 0;
  for (int a = tid; a < N; a += kAllocThreads) {
    double wgt = head_weight(inf, La, Ls, H, a, uniform);
    double q = __ddiv_rn(__dmul_rn((double)D, wgt), W);
    double fl = floor(q);
    rem[a] = __dadd_rn(q, -fl);
    long long f = (long long)fl;
    budgets[a] = (int32_t)f;                                          // floors for now
    fsum += f;
  }
  long long Rleft = D - block_sum_ll(fsum, red);
  if (Rleft >= N) {                                                   // not reachable in exact arithmetic
    long long each = Rleft / N;
    for (int a = tid; a < N; a += kAllocThreads) budgets[a] += (int32_t)each;
    Rleft -= each * N;
  }
  __syncthreads();
  if (Rleft > 0) {
    // largest remainder first, ties -> lower index: head a gets +1 iff fewer than Rleft heads precede it
    for (int a = tid; a < N; a += kAllocThreads) {
      double ra = rem[a];
      int rank = 0;
      for (int b = 0; b < N; ++b) {
        double rb = rem[b];
        rank += (rb > ra) || (rb == ra && b < a);
      }
      if (rank < Rleft) budgets[a] += 1;
    }
  }
  while (Rleft < 0) {
    // floors overshot D (rounding): take one back from the smallest remainders, ties -> higher index
    __syncthreads();
    long long taken = 0;
    int dec[(16384 + kAllocThreads - 1) / kAllocThreads];
    int nd = 0;
    for (int a = tid; a < N; a += kAllocThreads, ++nd) {
      dec[nd] = 0;
      if (budgets[a] <= 0) continue;
      double ra = rem[a];
      int rank = 0;
      for (int b = 0; b < N; ++b) {
        if (budgets[b] <= 0) continue;
        double rb = rem[b];
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

cudaError_t launch_alloc(const float* inf, int n_layers, int n_heads, int fixed, long long total, int32_t* budgets,
                         int32_t* status, cudaStream_t st) {
  size_t smem = (size_t)(n_layers * n_heads + n_layers) * sizeof(double);
  static thread_local int configured_dev = -1;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (configured_dev != dev) {
    e = cudaFuncSetAttribute(k_alloc, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    configured_dev = dev;
  }
  int launches = 0;
  LaunchScope scope(KID_ALLOC, st, &launches);
  k_alloc<<<1, kAllocThreads, smem, st>>>(inf, n_layers, n_heads, fixed, total, budgets, status);
  return cudaGetLastError();
}

}  // namespace slkv
