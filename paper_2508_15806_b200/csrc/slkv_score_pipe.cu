// Window relevance scores, two layers per launch (Sec. 3.4, Eq. 7; Algorithm 3; Eq. 3-4): pass 1 (row statistics)
// of one layer and pass 2 (votes) of the layer before it run side by side in every CTA.
//
// The softmax over the keys needs every key of a row before any vote can be formed, so one layer's two passes
// cannot overlap -- but consecutive layers are independent.  A launch therefore carries two streams of 128-key
// tiles over the same split (one CTA per SM):
//   stream A  pass 1 of layer n:     S = Q K^T, a TMEM lane owns a query row, per-CTA (max, sum) partials out;
//   stream B  pass 2 of layer n - 1: S^T = K Q^T, a TMEM lane owns a key; the row log-sum-exps come from the
//             partials the launch before this one wrote, so the launch boundary is the grid-wide barrier.
// Each stream has its own TMA producer thread, MMA issuer thread, K ring, Q tile, two TMEM accumulators and two
// epilogue warpgroups; the special-function and FMA pipes, which bound both passes, never wait for one stream's
// barrier, merge, ramp-up or load latency while the other has tiles ready.
// Shapes: bf16, head_dim 128, G * w <= 128 query rows per KV head.  Every wait is bounded (1 s), as in the
// single-layer kernels: SLKV_ERR_DEVICE_TIMEOUT in the status words, TMEM freed, return.
#include <cuda.h>

#include "slkv_internal.cuh"
#include "slkv_tc_device.cuh"

namespace slkv {
namespace {

constexpr int kPipeThreads = 640;        // warps 0-3: producer A, issuer A, producer B, issuer B;
                                         // warps 4-11: epilogue of stream A; warps 12-19: epilogue of stream B
constexpr int kStagesA = 3;              // K tiles in flight from HBM
constexpr int kStagesB = 2;              // K tiles in flight from L2
constexpr int kQBytes = 2 * kHalfBytes;  // one 128-row Q tile
constexpr int kBarBytesPerStream = 128;  // up to 16 mbarriers
constexpr int kPipeTail = 512 + 1024 + 1024;   // mbarriers + flags, stat_m/stat_z of stream A, two log-sum-exp rows of stream B
constexpr int kPipeSmem = 2 * kQBytes + (kStagesA + kStagesB) * kStageBytes + kPipeTail;
static_assert(kPipeSmem <= kSmemLimit, "shared memory of the two-stream kernel");

struct PipeArgs {
  TcArgs a;        // stream A: pass 1 of this layer
  TcArgs b;        // stream B: pass 2 of this layer
  int has_a, has_b;
};

// One stream's resources inside the CTA.
struct StreamCtx {
  uint32_t q_smem, k_smem, bar0, tmem0;
  int n_stages, begin, end;
  volatile int* abort_flag;
  __device__ __forceinline__ uint32_t full_bar(int st) const { return bar0 + 8u * st; }
  __device__ __forceinline__ uint32_t empty_bar(int st) const { return bar0 + 8u * (3 + st); }
  __device__ __forceinline__ uint32_t accf_bar(int b) const { return bar0 + 8u * (6 + b); }
  __device__ __forceinline__ uint32_t acce_bar(int b) const { return bar0 + 8u * (8 + b); }
  __device__ __forceinline__ uint32_t qfull_bar() const { return bar0 + 8u * 10; }
  __device__ __forceinline__ uint32_t qempty_bar() const { return bar0 + 8u * 11; }
};

__device__ __forceinline__ void named_bar(int id) { asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(kEpiThreads) : "memory"); }

// ---- one thread: TMA loads of the stream's Q tiles and K tiles ------------------------------------------
template <bool REV>
__device__ __forceinline__ void producer(const StreamCtx& c, const TcArgs& a, const CUtensorMap* tm_q, const CUtensorMap* tm_k) {
  int it = 0, run_idx = 0, st = 0;
  uint32_t st_phase = 0;
  bool ok = true;
  for (int pos = REV ? c.end - 1 : c.begin; (REV ? pos >= c.begin : pos < c.end) && ok;) {
    const Run r = locate(a, pos, c.begin, c.end, REV);
    ok = mbar_wait(c.qempty_bar(), (run_idx & 1) ^ 1, c.abort_flag);        // the run before is done with Q
    if (!ok) break;
    mbar_expect_tx(c.qfull_bar(), 2u * (uint32_t)a.R * 128u);
    const int qy = a.q_head_inner ? r.g * a.G : 0, qz = a.q_head_inner ? 0 : r.g * a.G;
    tma_load_4d(c.q_smem, tm_q, 0, qy, qz, r.s, c.qfull_bar());
    tma_load_4d(c.q_smem + kHalfBytes, tm_q, 64, qy, qz, r.s, c.qfull_bar());
    int tok = a.tab.cu_at(r.s) + (r.t0 + (REV ? r.count - 1 : 0)) * kTileKeys;
    const int tok_step = REV ? -kTileKeys : kTileKeys;
    for (int i = 0; i < r.count; ++i, ++it, tok += tok_step) {
      ok = mbar_wait(c.empty_bar(st), st_phase ^ 1u, c.abort_flag);
      if (!ok) break;
      const uint32_t fb = c.full_bar(st), dst = c.k_smem + (uint32_t)st * kStageBytes;
      mbar_expect_tx(fb, kStageBytes);
      const int ky = a.k_head_inner ? r.g : tok, kz = a.k_head_inner ? tok : r.g;
      tma_load_3d(dst, tm_k, 0, ky, kz, fb);
      tma_load_3d(dst + kHalfBytes, tm_k, 64, ky, kz, fb);
      if (++st == c.n_stages) { st = 0; st_phase ^= 1u; }
    }
    pos = REV ? pos - r.count : pos + r.count;
    ++run_idx;
  }
  if (!ok) {
    // give loads already in flight a bounded chance to land before the CTA's shared memory goes away
    const unsigned long long t0 = now_ns();
    for (int s2 = 0; s2 < c.n_stages; ++s2) {
      const int last = it - 1 - ((it - 1 - s2) % c.n_stages + c.n_stages) % c.n_stages;   // last issue into stage s2
      if (it == 0 || last < 0) continue;
      while (!mbar_try(c.full_bar(s2), (last / c.n_stages) & 1) && now_ns() - t0 < kWaitLimitNs) {}
    }
  }
}

// ---- one thread: the stream's MMAs, one 128 x 128 x 128 product per tile into one of two accumulators --------
template <bool REV>
__device__ __forceinline__ void issuer(const StreamCtx& c, const TcArgs& a) {
  // pass 1: D[row, key] = Q K^T (A = Q, B = K); pass 2: D[key, row] = K Q^T (A = K, B = Q, N = R)
  const uint32_t idesc = REV ? instr_desc(kTileKeys, a.R) : instr_desc(128, kTileKeys);
  const uint64_t q_desc0 = smem_desc(c.q_smem), k_desc0 = smem_desc(c.k_smem);
  const uint64_t hi = (uint64_t)(kHalfBytes >> 4);
  int it = 0, run_idx = 0, st = 0, b = 0;
  uint32_t st_phase = 0, b_phase = 0;
  uint64_t k_desc = k_desc0;
  bool ok = true;
  for (int pos = REV ? c.end - 1 : c.begin; (REV ? pos >= c.begin : pos < c.end) && ok;) {
    const Run r = locate(a, pos, c.begin, c.end, REV);
    ok = mbar_wait(c.qfull_bar(), run_idx & 1, c.abort_flag);
    if (!ok) break;
    for (int i = 0; i < r.count; ++i, ++it) {
      ok = mbar_wait(c.full_bar(st), st_phase, c.abort_flag) && mbar_wait(c.acce_bar(b), b_phase ^ 1u, c.abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t d0 = c.tmem0 + (uint32_t)(b * 128);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const uint64_t off = (uint64_t)((ks & 3) * 2) + (ks >> 2) * hi;
        if (REV) tc_mma(d0, k_desc + off, q_desc0 + off, idesc, ks > 0);
        else tc_mma(d0, q_desc0 + off, k_desc + off, idesc, ks > 0);
      }
      tc_commit(c.empty_bar(st));       // K stage free once these MMAs have read it
      tc_commit(c.accf_bar(b));         // accumulator ready for the epilogue
      k_desc += (uint64_t)(kStageBytes >> 4);
      if (++st == c.n_stages) { st = 0; st_phase ^= 1u; k_desc = k_desc0; }
      if (++b == 2) { b = 0; b_phase ^= 1u; }
    }
    tc_commit(c.qempty_bar());          // Q tile free once the run's MMAs are done
    pos = REV ? pos - r.count : pos + r.count;
    ++run_idx;
  }
}

// ---- 256 threads: pass 1, row statistics (stream A) ----------------------------------------------------------
__device__ __forceinline__ void epilogue_rows(const StreamCtx& c, const TcArgs& a, int et, int warp, float* stat_m, float* stat_z) {
  const int wg = et >> 7, row = et & 127, lane = et & 31;
  const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
  const float sc = a.scale_log2;
  const int R = a.R;
  int it = 0;
  bool ok = true;
  for (int pos = c.begin; pos < c.end;) {
    const Run r = locate(a, pos, c.begin, c.end, false);
    const int seg = r.s * a.n_kv_heads + r.g;
    const int first_cta = r.seg_tile0 / a.tiles_per_cta;
    float m = 0.f, z = 0.f;                                   // fixed reference 0 on the fast path
    for (int i = 0; i < r.count; ++i, ++it) {
      if ((it & 1) != wg) continue;
      const int b = it & 1;
      if (ok) ok = mbar_wait(c.accf_bar(b), (it >> 1) & 1, c.abort_flag);
      ok = __all_sync(0xffffffffu, ok) != 0;                  // the TMEM loads below need the whole warp
      if (!ok) continue;
      tc_fence_after();
      if (et == 0 && it == 0) trace_mark(a.trace, 2);
      const int key0 = (r.t0 + i) * kTileKeys;
      const int n_valid = min(r.n_hist - key0, kTileKeys);
      const uint32_t tcol = c.tmem0 + lane_sel + (uint32_t)(b * 128);
      // A fixed reference m per row (0 until a fallback moves it) instead of a running maximum: any reference gives
      // the same log-sum-exp as long as nothing overflows and not everything underflows.  A chunk whose sum is not
      // finite and positive is redone exactly from the registers, which moves the reference.  Keys past the
      // segment's end (its ragged last tile) are left out chunk by chunk.
      uint32_t ra[32], rb[32];
      auto add_chunk = [&](const uint32_t (&rr)[32], int nv) {
        if (nv >= 32) {
          const float zc = sum_ex2_32(rr, sc, m);
          const float zn = z + zc;
          if (zn < INFINITY && zc > 0.f) { z = zn; return; }
        }
        // rare: a copy goes through the stack so that the chunk registers themselves never have to
        uint32_t tmp[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) tmp[e] = rr[e];
        chunk_stats_exact(tmp, sc, nv < 32 ? nv : 32, m, z);
      };
      tc_ld32_issue(tcol, ra);
#pragma unroll 1
      for (int c0 = 0; c0 < kTileKeys; c0 += 64) {
        const bool last = c0 + 64 >= kTileKeys;
        tc_ld_wait(ra);
        tc_ld32_issue(tcol + c0 + 32, rb);
        if (last) {
          // the whole accumulator is in registers (or on its way): hand the TMEM buffer back before the arithmetic
          tc_ld_wait(rb);
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(c.acce_bar(b));
        }
        add_chunk(ra, n_valid - c0);
        if (!last) {
          tc_ld_wait(rb);
          tc_ld32_issue(tcol + c0 + 64, ra);
        }
        add_chunk(rb, n_valid - c0 - 32);
      }
    }
    // combine the two warpgroups' statistics and publish this CTA's partial for the segment
    const int slot = blockIdx.x - first_cta;
    if (wg == 1) { stat_m[row] = m; stat_z[row] = z; }
    named_bar(1);
    if (wg == 0 && row < R) {
      const float m1 = stat_m[row], z1 = stat_z[row];
      const bool h0 = z > 0.f, h1 = z1 > 0.f;                  // a warpgroup without a tile in this run has z = 0
      const float M = h0 && h1 ? fmaxf(m, m1) : (h0 ? m : m1);
      float Z = 0.f;
      if (h0) Z += z * ex2(m - M);
      if (h1) Z += z1 * ex2(m1 - M);
      a.part_m[((long long)seg * a.slot_stride + slot) * R + row] = M;
      a.part_z[((long long)seg * a.slot_stride + slot) * R + row] = Z;
    }
    named_bar(1);
    pos += r.count;
  }
}

// sum_e 2^(v_e * sc - lse_e) over 32 accumulator values (32 query rows of one key)
__device__ __forceinline__ float vote_chunk(const uint32_t (&r)[32], float sc, const float* lse) {
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
  for (int e = 0; e < 32; e += 4) {
    const float4 l4 = *reinterpret_cast<const float4*>(lse + e);
    s0 += ex2(fmaf(__uint_as_float(r[e]), sc, -l4.x));
    s1 += ex2(fmaf(__uint_as_float(r[e + 1]), sc, -l4.y));
    s2 += ex2(fmaf(__uint_as_float(r[e + 2]), sc, -l4.z));
    s3 += ex2_fma(fmaf(__uint_as_float(r[e + 3]), sc, -l4.w), false);
  }
  return (s0 + s1) + (s2 + s3);
}

// ---- 256 threads: pass 2, votes (stream B) ---------------------------------------------------------------------
__device__ __forceinline__ void epilogue_votes(const StreamCtx& c, const TcArgs& a, int et, int warp, float* lse2) {
  const int wg = et >> 7, row = et & 127, lane = et & 31;
  const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
  const float sc = a.scale_log2;
  const float inv_g = 1.0f / (float)a.G;
  const int R = a.R;
  int it = 0, run_idx = 0;
  bool ok = true;
  for (int pos = c.end - 1; pos >= c.begin;) {
    const Run r = locate(a, pos, c.begin, c.end, true);
    const int seg = r.s * a.n_kv_heads + r.g;
    const int first_cta = r.seg_tile0 / a.tiles_per_cta;
    float* lse = lse2 + 128 * (run_idx & 1);
    {
      // merge the per-CTA partials of this segment into the rows' log-sum-exp (log2 units): two neighbouring
      // lanes share a row (even / odd slots), all loads in flight before the first use
      const int n_slots = (r.seg_tile0 + r.tiles_seg - 1) / a.tiles_per_cta - first_cta + 1;
      const int rr = (et >> 1) < R ? (et >> 1) : -1;
      const int half = et & 1;
      float M = -INFINITY, Z = 0.f;
      if (rr >= 0) {
        const float* pm = a.part_m + (long long)seg * a.slot_stride * R + rr;      // [segment][slot][row]
        const float* pz = a.part_z + (long long)seg * a.slot_stride * R + rr;
        for (int c0 = half; c0 < n_slots; c0 += 24) {
          float m12[12], z12[12];
#pragma unroll
          for (int u = 0; u < 12; ++u) {
            const int cc = c0 + u * 2;
            const bool in = cc < n_slots;
            m12[u] = in ? __ldcg(pm + (long long)cc * R) : -INFINITY;
            z12[u] = in ? __ldcg(pz + (long long)cc * R) : 0.f;
          }
#pragma unroll
          for (int u = 0; u < 12; ++u)
            if (z12[u] > 0.f) {                                       // empty partials carry z = 0
              const float Mn = fmaxf(M, m12[u]);
              Z = Z * ex2(M - Mn) + z12[u] * ex2(m12[u] - Mn);      // ex2(-inf) = 0 covers the first term
              M = Mn;
            }
        }
      }
      const float M1 = __shfl_xor_sync(0xffffffffu, M, 1), Z1 = __shfl_xor_sync(0xffffffffu, Z, 1);
      const float Mn = fmaxf(M, M1);
      float Zt = 0.f;
      if (M > -INFINITY) Zt += Z * ex2(M - Mn);
      if (M1 > -INFINITY) Zt += Z1 * ex2(M1 - Mn);
      if (half == 0 && rr >= 0) lse[rr] = Mn + log2f(Zt);
    }
    named_bar(2);
    if (et == 0 && run_idx == 0) trace_mark(a.trace, 3);
    for (int i = 0; i < r.count; ++i, ++it) {
      if ((it & 1) != wg) continue;
      const int b = it & 1;
      if (ok) ok = mbar_wait(c.accf_bar(b), (it >> 1) & 1, c.abort_flag);
      ok = __all_sync(0xffffffffu, ok) != 0;
      if (!ok) continue;
      tc_fence_after();
      const int key0 = (r.t0 + r.count - 1 - i) * kTileKeys;
      const uint32_t tb = c.tmem0 + lane_sel + (uint32_t)(b * 128);
      uint32_t ra[32], rb[32];
      float acc = 0.f;
      auto release = [&]() {
        // the accumulator is in registers: hand its TMEM buffer back before the arithmetic and the vote's store
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(c.acce_bar(b));
      };
      tc_ld32_issue(tb, ra);
#pragma unroll 1
      for (int c0 = 0; c0 < R; c0 += 64) {
        tc_ld_wait(ra);
        if (c0 + 32 < R) tc_ld32_issue(tb + c0 + 32, rb);
        if (c0 + 32 >= R) release();
        else if (c0 + 64 >= R) { tc_ld_wait(rb); release(); }
        acc += vote_chunk(ra, sc, lse + c0);
        if (c0 + 32 < R) {
          if (c0 + 64 < R) { tc_ld_wait(rb); tc_ld32_issue(tb + c0 + 64, ra); }
          acc += vote_chunk(rb, sc, lse + c0 + 32);
        }
      }
      const int j = key0 + row;
      if (j < r.n_hist) a.vote[a.tab.hist_at(r.s) * a.n_kv_heads + (long long)r.g * r.n_hist + j] = acc * inv_g;
    }
    pos -= r.count;
    ++run_idx;
  }
}

__global__ void __launch_bounds__(kPipeThreads, 1)
k_score_pipe(const __grid_constant__ CUtensorMap tm_qa, const __grid_constant__ CUtensorMap tm_ka,
             const __grid_constant__ CUtensorMap tm_qb, const __grid_constant__ CUtensorMap tm_kb,
             const __grid_constant__ PipeArgs pa) {
  // Shared memory, all dynamic and 1024-byte aligned (the swizzled tiles need it):
  //   [Q of A 32 KB][Q of B 32 KB][K ring of A 3 x 32 KB][K ring of B 2 x 32 KB][mbarriers, flags 512 B]
  //   [stat_m, stat_z of A 1 KB][log-sum-exp rows of B 2 x 512 B]
  extern __shared__ __align__(1024) unsigned char smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  unsigned char* tail = smem + 2 * kQBytes + (kStagesA + kStagesB) * kStageBytes;
  uint32_t& tmem_base_sh = *reinterpret_cast<uint32_t*>(tail + 256);
  int& abort_sh = *reinterpret_cast<int*>(tail + 260);
  float* stat_m = reinterpret_cast<float*>(tail + 512);
  float* stat_z = stat_m + 128;
  float* lse2 = stat_m + 256;
  const bool has_a = pa.has_a != 0, has_b = pa.has_b != 0;
  int32_t* status_a = has_a ? pa.a.status : nullptr;
  int32_t* status_b = has_b ? pa.b.status : nullptr;
  if ((smem_u32(smem) & 1023u) != 0) {                      // never run on a skewed layout (uniform over the CTA)
    if (tid == 0 && status_a) atomicExch(status_a, (int)SLKV_ERR_BAD_ALIGN);
    if (tid == 0 && status_b) atomicExch(status_b, (int)SLKV_ERR_BAD_ALIGN);
    return;
  }
  StreamCtx ca, cb;
  ca.q_smem = smem_u32(smem);
  cb.q_smem = ca.q_smem + kQBytes;
  ca.k_smem = ca.q_smem + 2 * kQBytes;
  cb.k_smem = ca.k_smem + kStagesA * kStageBytes;
  ca.bar0 = smem_u32(tail);
  cb.bar0 = ca.bar0 + kBarBytesPerStream;
  ca.n_stages = kStagesA;
  cb.n_stages = kStagesB;
  ca.abort_flag = cb.abort_flag = &abort_sh;
  ca.begin = has_a ? min(blockIdx.x * pa.a.tiles_per_cta, pa.a.total_tiles) : 0;
  ca.end = has_a ? min(ca.begin + pa.a.tiles_per_cta, pa.a.total_tiles) : 0;
  cb.begin = has_b ? min(blockIdx.x * pa.b.tiles_per_cta, pa.b.total_tiles) : 0;
  cb.end = has_b ? min(cb.begin + pa.b.tiles_per_cta, pa.b.total_tiles) : 0;

  unsigned long long* trace = has_a ? pa.a.trace : pa.b.trace;
  if (tid == 0) trace_mark(trace, 0);
  if (tid == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_ka)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_kb)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_qa)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_qb)) : "memory");
    abort_sh = 0;
    for (int s = 0; s < 2; ++s) {
      const StreamCtx& c = s ? cb : ca;
      for (int st = 0; st < 3; ++st) { mbar_init(c.full_bar(st), 1); mbar_init(c.empty_bar(st), 1); }
      for (int b = 0; b < 2; ++b) { mbar_init(c.accf_bar(b), 1); mbar_init(c.acce_bar(b), 4); }
      mbar_init(c.qfull_bar(), 1);
      mbar_init(c.qempty_bar(), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // rows of a Q tile beyond R are never written by TMA: keep them zero
  if ((has_a && pa.a.R != 128) || (has_b && pa.b.R != 128)) {
    for (int i = tid; i < 2 * kQBytes / 16; i += kPipeThreads) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_sh)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_sh;
  ca.tmem0 = tmem_base;
  cb.tmem0 = tmem_base + 256;
  pdl_launch_dependents();

  // Stream A reads this layer's Q and K for the first time and overwrites partials the launch before may still be
  // merging: all its roles wait for the work before this launch.  Stream B's loads and MMAs need only Q and K of
  // the layer before, which the launch before this one has read: they start at once; its epilogue needs that
  // launch's partials and waits.
  if (warp == 0) {
    if (lane == 0 && has_a) { pdl_wait(); producer<false>(ca, pa.a, &tm_qa, &tm_ka); }
  } else if (warp == 1) {
    if (lane == 0 && has_a) issuer<false>(ca, pa.a);
  } else if (warp == 2) {
    if (lane == 0 && has_b) producer<true>(cb, pa.b, &tm_qb, &tm_kb);
  } else if (warp == 3) {
    if (lane == 0 && has_b) issuer<true>(cb, pa.b);
  } else if (warp < 12) {
    if (has_a) {
      pdl_wait();
      if (tid == 128) trace_mark(trace, 1);
      epilogue_rows(ca, pa.a, tid - 128, warp, stat_m, stat_z);
      if (tid == 128) trace_mark(trace, 5);
    }
  } else {
    if (has_b) {
      pdl_wait();
      if (tid == 384) trace_mark(trace, 7);
      epilogue_votes(cb, pa.b, tid - 384, warp, lse2);
      if (tid == 384) trace_mark(trace, 6);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (abort_sh && tid == 0) {
    if (status_a) atomicExch(status_a, (int)SLKV_ERR_DEVICE_TIMEOUT);
    if (status_b) atomicExch(status_b, (int)SLKV_ERR_DEVICE_TIMEOUT);
  }
  if (tid == 0) trace_mark(trace, 4);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace

bool score_pipe_supported(const Problem& pb) {
  return tensor_path_supported(pb.p) && pb.R <= 128;
}

// One launch: pass 1 of plan `a` (or null) and pass 2 of plan `b` (or null).
cudaError_t launch_score_pipe(const TcPlan* a, const TcPlan* b, cudaStream_t st, int* launches) {
  const bool has_a = a && a->n_cta > 0, has_b = b && b->n_cta > 0;
  if (!has_a && !has_b) return cudaSuccess;
  static thread_local int configured_dev = -1;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (configured_dev != dev) {
    e = cudaFuncSetAttribute(k_score_pipe, cudaFuncAttributeMaxDynamicSharedMemorySize, kPipeSmem);
    if (e != cudaSuccess) return e;
    configured_dev = dev;
  }
  PipeArgs pa;
  const TcPlan* any = has_a ? a : b;
  pa.a = has_a ? a->a : any->a;
  pa.b = has_b ? b->a : any->a;
  pa.has_a = has_a; pa.has_b = has_b;
  int n_cta = 0;
  if (has_a) n_cta = a->n_cta;
  if (has_b && b->n_cta > n_cta) n_cta = b->n_cta;
  unsigned long long* tr = tensor_trace_buffer(0, n_cta);
  pa.a.trace = tr; pa.b.trace = tr;
  LaunchScope scope(KID_SCORE_PIPE, st, launches);
  return launch_pdl(k_score_pipe, dim3(n_cta), dim3(kPipeThreads), (size_t)kPipeSmem, st, 1,
                    has_a ? a->tm_q : any->tm_q, has_a ? a->tm_k : any->tm_k,
                    has_b ? b->tm_q : any->tm_q, has_b ? b->tm_k : any->tm_k, pa);
}

}  // namespace slkv
