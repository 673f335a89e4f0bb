// Attention behaviour analysis (Sec. 3.2, Algorithm 1): SF_sc, LG_sc and INF_sc of a batch of attention rows.
//
// One warp per row.  A row's needle positions N and top-k positions T arrive as index lists; the kernel reads only the
// weights at those positions (the rest of the row never matters), so a batch over [layers x heads x prompts] moves a
// few hundred bytes per row however long the context is.  Sets are sets: an index that occurs twice in a list counts
// once.  Sums are fp64 over at most a few hundred terms; 0 / 0 counts as 0.
#include "slkv_internal.cuh"

namespace slkv {
namespace {

constexpr int kRowsPerCta = 8;          // warps per CTA

__device__ __forceinline__ double warp_sum(double v) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__global__ void __launch_bounds__(kRowsPerCta * 32)
k_behavior(const float* __restrict__ attn, long long row_stride, int row_len, long long n_rows,
           const int32_t* __restrict__ needle_idx, int n_needle, long long needle_stride,
           const int32_t* __restrict__ topk_idx, int n_topk, long long topk_stride, float* __restrict__ sf,
           float* __restrict__ lg, float* __restrict__ inf) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * kRowsPerCta + (threadIdx.x >> 5);
  if (row >= n_rows) return;
  const float* W = attn + row * row_stride;
  const int32_t* Nn = needle_idx + row * needle_stride;
  const int32_t* Tt = topk_idx + row * topk_stride;
  auto valid = [&](int i) { return i >= 0 && i < row_len; };      // entries outside the row are padding
  // total needle weight TNW: every distinct needle position once
  double tnw = 0.0;
  for (int a = lane; a < n_needle; a += 32) {
    const int i = Nn[a];
    if (!valid(i)) continue;
    bool first = true;
    for (int b = 0; b < a; ++b) first = first && Nn[b] != i;
    if (first) tnw += (double)W[i];
  }
  // top-k positions: on a needle (WO, weight on target) or not (WD, weight that distracts)
  double wo = 0.0, wd = 0.0;
  for (int a = lane; a < n_topk; a += 32) {
    const int i = Tt[a];
    if (!valid(i)) continue;
    bool first = true;
    for (int b = 0; b < a; ++b) first = first && Tt[b] != i;
    if (!first) continue;
    bool on_needle = false;
    for (int b = 0; b < n_needle; ++b) on_needle = on_needle || Nn[b] == i;
    if (on_needle) wo += (double)W[i]; else wd += (double)W[i];
  }
  tnw = warp_sum(tnw); wo = warp_sum(wo); wd = warp_sum(wd);
  if (lane == 0) {
    const double ws = fmax(0.0, tnw - wo);                         // needle weight outside the top-k set
    const double s = wo + wd > 0.0 ? wo / (wo + wd) : 0.0;         // SF_sc: surface focus
    const double l = wo + ws > 0.0 ? wo / (wo + ws) : 0.0;         // LG_sc: logic grasp
    const double h = s + l > 0.0 ? 2.0 * s * l / (s + l) : 0.0;    // INF_sc: their harmonic mean
    sf[row] = (float)s; lg[row] = (float)l; inf[row] = (float)h;
  }
}

}  // namespace

cudaError_t launch_behavior(const float* attn, long long row_stride, int row_len, long long n_rows,
                            const int32_t* needle_idx, int n_needle, long long needle_stride, const int32_t* topk_idx,
                            int n_topk, long long topk_stride, float* sf, float* lg, float* inf, cudaStream_t st) {
  if (n_rows == 0) return cudaSuccess;
  int launches = 0;
  LaunchScope scope(KID_BEHAVIOR, st, &launches);
  const long long grid = (n_rows + kRowsPerCta - 1) / kRowsPerCta;
  return launch_pdl(k_behavior, dim3((unsigned)grid), dim3(kRowsPerCta * 32), 0, st, 1, attn, row_stride, row_len, n_rows,
                    needle_idx, n_needle, needle_stride, topk_idx, n_topk, topk_stride, sf, lg, inf);
}

}  // namespace slkv
