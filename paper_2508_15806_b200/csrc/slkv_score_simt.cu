// Window relevance scores with fp32 FMA arithmetic (Sec. 3.4, Eq. 7; Algorithm 3 l.6; Eq. 3-4).
//
// Serves the fp32 configuration and every shape the tensor-core kernels do not take.  One thread owns
// one history key (its row of K lives in registers), the G*w query rows of the KV head's group sit in
// shared memory, and a CTA walks a chunk of key tiles:
//   pass 1  per query row: running max and sum of 2^(s - max) over the chunk's keys -> part_m / part_z
//   pass 2  merges the chunks' partials into the row's log-sum-exp, then per key
//           vote[j] = (1/G) sum_rows 2^(s_rj - lse_r)      (s in log2 units: s = q.k * log2(e)/sqrt(d))
// The w x n_hist probability matrix never exists in memory.
#include "slkv_internal.cuh"

namespace slkv {
namespace {

constexpr int kThreads = 128;          // keys per tile
constexpr int kTilesPerChunk = 8;      // key tiles a CTA walks
constexpr int kRowBatch = 8;           // query rows reduced together in pass 1

template <typename T> struct Vec;      // 16-byte vector of T
template <> struct Vec<float> { static constexpr int N = 4; };
template <> struct Vec<__nv_bfloat16> { static constexpr int N = 8; };

__device__ __forceinline__ void unpack(const uint4& u, float (&f)[4], float) {
  f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y); f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
}
__device__ __forceinline__ void unpack(const uint4& u, float (&f)[8], __nv_bfloat16) {
  // a bf16 is the high half of an fp32
  f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xffff0000u);
  f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xffff0000u);
  f[4] = __uint_as_float(u.z << 16); f[5] = __uint_as_float(u.z & 0xffff0000u);
  f[6] = __uint_as_float(u.w << 16); f[7] = __uint_as_float(u.w & 0xffff0000u);
}

template <typename T, int D>
__device__ __forceinline__ float dot_row(const T* __restrict__ qrow /*smem*/, const float (&kreg)[D]) {
  constexpr int VN = Vec<T>::N;
  float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
  for (int c = 0; c < D / VN; ++c) {
    uint4 u = *reinterpret_cast<const uint4*>(qrow + c * VN);
    float f[VN];
    unpack(u, f, T());
#pragma unroll
    for (int e = 0; e < VN; e += 2) {
      acc0 = fmaf(f[e], kreg[c * VN + e], acc0);
      acc1 = fmaf(f[e + 1], kreg[c * VN + e + 1], acc1);
    }
  }
  return acc0 + acc1;
}

// Row log-sum-exp (log2 units) from the per-chunk statistics of the SIMT layout [row][chunk], the window keys'
// statistics folded in when there are any (softmax over all causally visible keys).
__device__ __forceinline__ float simt_row_lse(const float* pm, const float* pz, int nc, bool has_win, float wm,
                                              float wz) {
  float M = -INFINITY;
  for (int c = 0; c < nc; ++c) M = fmaxf(M, pm[c]);
  if (has_win) M = fmaxf(M, wm);
  float Z = 0.f;
  for (int c = 0; c < nc; ++c) Z = fmaf(pz[c], exp2f(pm[c] - M), Z);      // explicit rounding: the same in every kernel
  if (has_win) Z = fmaf(wz, exp2f(wm - M), Z);
  return __fadd_rn(M, log2f(Z));
}

template <typename T, int D, int PASS>
__global__ void __launch_bounds__(kThreads)
k_score_simt(const T* __restrict__ q, const T* __restrict__ k, const __grid_constant__ SeqTables tab,
             float* __restrict__ part_m, float* __restrict__ part_z,
             float* __restrict__ vote, const LseSource lse, int n_kv_heads, int G, int window, int n_chunks, long long k_stride_tok,
             long long k_stride_head, long long q_stride_seq, long long q_stride_row, long long q_stride_head,
             float scale_log2) {
  constexpr int VN = Vec<T>::N;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int R = G * window;
  T* qs = reinterpret_cast<T*>(smem_raw);                               // [R][D]
  float* fbuf = reinterpret_cast<float*>(smem_raw + (size_t)R * D * sizeof(T));
  float* run_m = fbuf;                                                  // [R]  (pass 2: lse per row)
  float* run_z = fbuf + R;                                              // [R]
  float* wred = fbuf + 2 * R;                                           // [2][kRowBatch][4]

  const int chunk = blockIdx.x, g = blockIdx.y, s = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  pdl_launch_dependents();
  pdl_wait();
  const int t0 = tab.cu_at(s);
  const int n_hist = max(tab.cu_at(s + 1) - t0 - window, 0);
  const int key0 = chunk * (kThreads * kTilesPerChunk);
  if (key0 >= n_hist) return;
  const int seg = s * n_kv_heads + g;

  // the group's query rows: row r = hh*window + i  <->  query head g*G + hh, window row i
  for (int idx = tid; idx < R * (D / VN); idx += kThreads) {
    int r = idx / (D / VN), c = idx - r * (D / VN);
    int hh = r / window, i = r - hh * window;
    const T* src = q + s * q_stride_seq + i * q_stride_row + (long long)(g * G + hh) * q_stride_head + c * VN;
    *reinterpret_cast<uint4*>(qs + r * D + c * VN) = *reinterpret_cast<const uint4*>(src);
  }
  if (PASS == 1) {
    for (int r = tid; r < R; r += kThreads) { run_m[r] = -INFINITY; run_z[r] = 0.f; }
  } else {
    const int nc = (n_hist + kThreads * kTilesPerChunk - 1) / (kThreads * kTilesPerChunk);
    for (int r = tid; r < R; r += kThreads) {
      if (lse.lse_opt) {                                                  // the caller's row statistics
        run_m[r] = lse.caller_lse(s, g, r, G, window, false);
        continue;
      }
      const float* pm = part_m + ((long long)seg * R + r) * n_chunks;
      const float* pz = part_z + ((long long)seg * R + r) * n_chunks;
      const bool has_win = lse.win_m != nullptr;
      run_m[r] = simt_row_lse(pm, pz, nc, has_win, has_win ? lse.win_m[(long long)seg * R + r] : 0.f,
                              has_win ? lse.win_z[(long long)seg * R + r] : 0.f);
    }
  }
  __syncthreads();

  for (int tile = 0; tile < kTilesPerChunk; ++tile) {
    const int j = key0 + tile * kThreads + tid;
    if (key0 + tile * kThreads >= n_hist) break;
    const bool valid = j < n_hist;
    float kreg[D];
    {
      const T* krow = k + (long long)(t0 + (valid ? j : 0)) * k_stride_tok + (long long)g * k_stride_head;
#pragma unroll
      for (int c = 0; c < D / VN; ++c) {
        uint4 u = *reinterpret_cast<const uint4*>(krow + c * VN);
        float f[VN];
        unpack(u, f, T());
#pragma unroll
        for (int e = 0; e < VN; ++e) kreg[c * VN + e] = f[e];
      }
    }
    if (PASS == 1) {
      for (int r0 = 0; r0 < R; r0 += kRowBatch) {
        float sv[kRowBatch], bm[kRowBatch];
#pragma unroll
        for (int b = 0; b < kRowBatch; ++b) {
          int r = min(r0 + b, R - 1);
          float d = dot_row<T, D>(qs + r * D, kreg) * scale_log2;
          sv[b] = valid ? d : -INFINITY;
          float m = sv[b];
          for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
          if (lane == 0) wred[b * 4 + wid] = m;
        }
        __syncthreads();
#pragma unroll
        for (int b = 0; b < kRowBatch; ++b) {
          bm[b] = fmaxf(fmaxf(wred[b * 4], wred[b * 4 + 1]), fmaxf(wred[b * 4 + 2], wred[b * 4 + 3]));
          float e = exp2f(sv[b] - bm[b]);
          for (int o = 16; o > 0; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
          if (lane == 0) wred[kRowBatch * 4 + b * 4 + wid] = e;
        }
        __syncthreads();
        if (tid < kRowBatch && r0 + tid < R) {
          const int r = r0 + tid;
          const float* ws = wred + kRowBatch * 4 + tid * 4;
          float bs = (ws[0] + ws[1]) + (ws[2] + ws[3]);
          const float* wm = wred + tid * 4;                 // the batch's warp maxima are still in place
          float tm = fmaxf(fmaxf(wm[0], wm[1]), fmaxf(wm[2], wm[3]));
          float om = run_m[r], nm = fmaxf(om, tm);
          run_z[r] = run_z[r] * exp2f(om - nm) + bs * exp2f(tm - nm);
          run_m[r] = nm;
        }
        __syncthreads();
      }
    } else {
      float acc = 0.f;
      for (int r = 0; r < R; ++r) acc += exp2f(dot_row<T, D>(qs + r * D, kreg) * scale_log2 - run_m[r]);
      if (valid) vote[tab.hist_at(s) * n_kv_heads + (long long)g * n_hist + j] = acc / (float)G;
    }
  }
  if (PASS == 1) {
    __syncthreads();
    for (int r = tid; r < R; r += kThreads) {
      part_m[((long long)seg * R + r) * n_chunks + chunk] = run_m[r];
      part_z[((long long)seg * R + r) * n_chunks + chunk] = run_z[r];
    }
  }
}

// Row statistics over the window keys a window row sees causally (its own position and the window keys before it):
// one CTA per segment, one thread per row.  Only the all-causal softmax domain needs them.
template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
k_window_stats(const T* __restrict__ q, const T* __restrict__ k, const __grid_constant__ SeqTables tab,
               float* __restrict__ win_m, float* __restrict__ win_z, int n_kv_heads, int G, int window, int head_inner,
               long long k_stride_tok, long long k_stride_head, long long q_stride_seq, long long q_stride_row,
               long long q_stride_head, float scale_log2) {
  constexpr int VN = Vec<T>::N;
  pdl_launch_dependents();
  pdl_wait();
  const int seg = blockIdx.x, s = seg / n_kv_heads, g = seg - s * n_kv_heads;
  const int t0 = tab.cu_at(s);
  const int n_hist = tab.cu_at(s + 1) - t0 - window;
  if (n_hist <= 0) return;                                   // no history: nothing is scored
  const int R = G * window;
  for (int r = threadIdx.x; r < R; r += kThreads) {
    const int hh = head_inner ? r % G : r / window;
    const int i = head_inner ? r / G : r - hh * window;
    const T* qrow = q + s * q_stride_seq + i * q_stride_row + (long long)(g * G + hh) * q_stride_head;
    float m = -INFINITY, z = 0.f;
    for (int j = 0; j <= i; ++j) {                           // window key j is token n_hist + j
      const T* krow = k + (long long)(t0 + n_hist + j) * k_stride_tok + (long long)g * k_stride_head;
      float acc0 = 0.f, acc1 = 0.f;
      for (int c = 0; c < D / VN; ++c) {
        float fq[VN], fk[VN];
        unpack(*reinterpret_cast<const uint4*>(qrow + c * VN), fq, T());
        unpack(*reinterpret_cast<const uint4*>(krow + c * VN), fk, T());
#pragma unroll
        for (int e = 0; e < VN; e += 2) {
          acc0 = fmaf(fq[e], fk[e], acc0);
          acc1 = fmaf(fq[e + 1], fk[e + 1], acc1);
        }
      }
      const float x = (acc0 + acc1) * scale_log2;
      const float mn = fmaxf(m, x);
      z = z * exp2f(m - mn) + exp2f(x - mn);                 // exp2f(-inf) = 0 covers the first key
      m = mn;
    }
    win_m[(long long)seg * R + r] = m;
    win_z[(long long)seg * R + r] = z;
  }
}

// lse_out[s][h][i] from the SIMT layout's per-chunk statistics (and the window statistics, if any).
__global__ void __launch_bounds__(kThreads)
k_merge_lse_simt(const float* __restrict__ part_m, const float* __restrict__ part_z, const LseSource lse,
                 const __grid_constant__ SeqTables tab, float* __restrict__ lse_out, int n_kv_heads, int G, int window,
                 int n_chunks, int chunk_keys, float out_scale) {
  pdl_launch_dependents();
  pdl_wait();
  const int seg = blockIdx.x, s = seg / n_kv_heads, g = seg - s * n_kv_heads;
  const int n_hist = tab.cu_at(s + 1) - tab.cu_at(s) - window;
  if (n_hist <= 0) return;
  const int R = G * window;
  const int nc = (n_hist + chunk_keys - 1) / chunk_keys;
  for (int r = threadIdx.x; r < R; r += kThreads) {
    const float* pm = part_m + ((long long)seg * R + r) * n_chunks;
    const float* pz = part_z + ((long long)seg * R + r) * n_chunks;
    const bool has_win = lse.win_m != nullptr;
    const float l2 = simt_row_lse(pm, pz, nc, has_win, has_win ? lse.win_m[(long long)seg * R + r] : 0.f,
                                  has_win ? lse.win_z[(long long)seg * R + r] : 0.f);
    const int hh = r / window, i = r - hh * window;
    lse_out[((long long)s * lse.n_q_heads + g * G + hh) * window + i] = l2 * out_scale;
  }
}

template <typename T, int D>
cudaError_t launch_passes(const Problem& pb, int passes, cudaStream_t st, int* launches) {
  const size_t smem = simt_smem_bytes(pb);
  static thread_local int configured_dev = -1;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (configured_dev != dev) {
    e = cudaFuncSetAttribute(k_score_simt<T, D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_score_simt<T, D, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    configured_dev = dev;
  }
  const int chunk_keys = kThreads * kTilesPerChunk;
  dim3 grid((pb.max_hist + chunk_keys - 1) / chunk_keys, pb.p.n_kv_heads, pb.p.n_seqs);
  const float scale_log2 = kLog2e / sqrtf((float)pb.p.head_dim);
  const slkv_params& p = pb.p;
  const LseSource lse = lse_source_of(pb);
  if (passes & 1) {
    LaunchScope scope(KID_SCORE_LSE, st, launches);
    e = launch_pdl(k_score_simt<T, D, 1>, grid, dim3(kThreads), smem, st, 1, (const T*)pb.q, (const T*)pb.k, pb.tab,
                   pb.part_m, pb.part_z, pb.vote, lse, p.n_kv_heads, pb.G, p.window, pb.n_chunks,
                   (long long)p.k_stride_tok, (long long)p.k_stride_head, (long long)p.q_stride_seq,
                   (long long)p.q_stride_row, (long long)p.q_stride_head, scale_log2);
    if (e != cudaSuccess) return e;
  }
  if (!(passes & 2)) return cudaSuccess;
  LaunchScope scope(KID_SCORE_VOTE, st, launches);
  return launch_pdl(k_score_simt<T, D, 2>, grid, dim3(kThreads), smem, st, 1, (const T*)pb.q, (const T*)pb.k, pb.tab,
                    pb.part_m, pb.part_z, pb.vote, lse, p.n_kv_heads, pb.G, p.window, pb.n_chunks,
                    (long long)p.k_stride_tok, (long long)p.k_stride_head, (long long)p.q_stride_seq,
                    (long long)p.q_stride_row, (long long)p.q_stride_head, scale_log2);
}

template <typename T, int D>
cudaError_t launch_window(const Problem& pb, bool head_inner, cudaStream_t st, int* launches) {
  const slkv_params& p = pb.p;
  LaunchScope scope(KID_WINDOW_STATS, st, launches);
  return launch_pdl(k_window_stats<T, D>, dim3(pb.n_seg), dim3(kThreads), 0, st, 1, (const T*)pb.q, (const T*)pb.k,
                    pb.tab, pb.win_m, pb.win_z, p.n_kv_heads, pb.G, p.window, head_inner ? 1 : 0,
                    (long long)p.k_stride_tok, (long long)p.k_stride_head, (long long)p.q_stride_seq,
                    (long long)p.q_stride_row, (long long)p.q_stride_head, kLog2e / sqrtf((float)p.head_dim));
}

}  // namespace

int simt_chunk_keys() { return kThreads * kTilesPerChunk; }

size_t simt_smem_bytes(const Problem& pb) {
  return (size_t)pb.R * pb.p.head_dim * pb.elem + (size_t)(2 * pb.R + 2 * kRowBatch * 4) * sizeof(float);
}

cudaError_t launch_score_simt(const Problem& pb, int passes, cudaStream_t st, int* launches) {
  if (pb.max_hist <= 0) return cudaSuccess;
  const bool bf = pb.p.dtype == SLKV_BF16;
  if (pb.p.head_dim == 64)
    return bf ? launch_passes<__nv_bfloat16, 64>(pb, passes, st, launches) : launch_passes<float, 64>(pb, passes, st, launches);
  return bf ? launch_passes<__nv_bfloat16, 128>(pb, passes, st, launches) : launch_passes<float, 128>(pb, passes, st, launches);
}

cudaError_t launch_window_stats(const Problem& pb, bool head_inner, cudaStream_t st, int* launches) {
  if (pb.max_hist <= 0) return cudaSuccess;
  const bool bf = pb.p.dtype == SLKV_BF16;
  if (pb.p.head_dim == 64)
    return bf ? launch_window<__nv_bfloat16, 64>(pb, head_inner, st, launches) : launch_window<float, 64>(pb, head_inner, st, launches);
  return bf ? launch_window<__nv_bfloat16, 128>(pb, head_inner, st, launches) : launch_window<float, 128>(pb, head_inner, st, launches);
}

// The row statistics a vote pass (or the merge) uses besides the partials of its own pass 1.
LseSource lse_source_of(const Problem& pb) {
  LseSource l;
  l.lse_opt = pb.lse_opt;
  const bool win = !pb.lse_opt && pb.p.softmax_domain == SLKV_ALL_CAUSAL;
  l.win_m = win ? pb.win_m : nullptr;
  l.win_z = win ? pb.win_z : nullptr;
  l.to_log2 = pb.p.lse_units == SLKV_LSE_LOG2 ? 1.0f : kLog2e;
  l.n_q_heads = pb.p.n_q_heads;
  return l;
}

float lse_out_scale(const Problem& pb) { return pb.p.lse_units == SLKV_LSE_LOG2 ? 1.0f : 0.6931471805599453f; }

cudaError_t launch_merge_lse_simt(const Problem& pb, float* lse_out, cudaStream_t st, int* launches) {
  if (pb.max_hist <= 0) return cudaSuccess;
  LaunchScope scope(KID_MERGE_LSE, st, launches);
  return launch_pdl(k_merge_lse_simt, dim3(pb.n_seg), dim3(kThreads), 0, st, 1, (const float*)pb.part_m,
                    (const float*)pb.part_z, lse_source_of(pb), pb.tab, lse_out, pb.p.n_kv_heads, pb.G, pb.p.window,
                    pb.n_chunks, pb.chunk_keys, lse_out_scale(pb));
}

}  // namespace slkv
