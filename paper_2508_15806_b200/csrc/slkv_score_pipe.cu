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
// A launch takes a list of layers: stream A walks pass 1 of layers 1..n, stream B pass 2 of layers 0..n-1 (layer 0
// is the one whose pass 1 the launch before did) or 0..n.  Pass 2 of a layer of the same launch waits until every
// CTA has published that layer's row statistics (one counter per layer, all CTAs resident: cooperative launch);
// stream A never waits for anything, so the ramp-up, the launch gap and the stragglers of a launch are paid once per
// list, not once per layer.
// Shapes: bf16, head_dim 128, G * w <= 128 query rows per KV head.  Every wait is bounded (1 s), as in the
// single-layer kernels: SLKV_ERR_DEVICE_TIMEOUT in the status words, TMEM freed, return.
#include <cuda.h>

#include <atomic>
#include <cstdlib>
#include <cstring>

#include "slkv_internal.cuh"
#include "slkv_tc_device.cuh"

namespace slkv {
namespace {

constexpr int kPipeThreads = 640;        // warps 0-3: producer A, issuer A, producer B, issuer B;
                                         // warps 4-11: epilogue of stream A; warps 12-19: epilogue of stream B
constexpr int kDualWgs = 3;               // vote pass on both streams: warpgroups per stream
constexpr int kDualThreads = 128 + 2 * kDualWgs * 128;
constexpr int kLeadEntries = 2;           // entries pass 1 may be ahead of the entry pass 2 has begun
constexpr unsigned kPollNs = 64;          // pause between two polls of an mbarrier
constexpr int kStagesA = 2;              // K tiles in flight for stream A (pass 1: first read of a layer's K)
constexpr int kStagesB = 3;              // ... for stream B (pass 2: ~70 % of its re-reads come from HBM again, and
                                         // its tiles take longer; measured 1.7 % faster than 3 + 2)
constexpr int kQBytes = 2 * kHalfBytes;  // one 128-row Q tile
constexpr int kBarBytesPerStream = 160;  // up to 20 mbarriers
constexpr int kPipeTail = 512 + 1024 + 1024;   // mbarriers + flags, stat_m/stat_z of stream A, two log-sum-exp rows of stream B
constexpr int kPipeSmem = 2 * kQBytes + (kStagesA + kStagesB) * kStageBytes + kPipeTail;
static_assert(kPipeSmem <= kSmemLimit, "shared memory of the two-stream kernel");

// Entries a layer may be split into (1 or 2).  Two halves the K that lies between pass 1 and pass 2, and pass 2 then
// finds it in L2 (measured: 299 B of DRAM traffic per key row instead of 442, SM clock 1.82 instead of 1.64 GHz under
// the power cap) but pays for twice the merges, Q reloads and waits for the other CTAs: 35.7 against 34.3 us per
// layer.  One it is.
constexpr int kMaxGroups = 1;
constexpr int kMaxLay = kPipeMaxLayers * kMaxGroups + 1;   // the entry pending from the launch before + this launch's
constexpr int kCountWords = kMaxLay + 1;        // per launch: one publish counter per layer + one exit counter
constexpr int kCountSlots = 64;                 // launches whose counters are live at once

// One entry of a launch's list: a layer, or one group of consecutive segments of a layer (a range of the layer's
// flat tile list).  Smaller entries keep less K between pass 1 and pass 2.
struct LayerDesc {
  alignas(64) CUtensorMap tm_q;
  alignas(64) CUtensorMap tm_k;
  float* part_m;
  float* part_z;
  float* vote;
  LseSource lse;               // where pass 2 takes the rows' log-sum-exp from besides this launch's / the last launch's pass 1
  int32_t* status;
  int tile_begin, tile_end;    // the entry's tiles in the layer's tile list; CTA b takes tiles_per_cta of them from
                               // tile_begin + b * tiles_per_cta
};
struct PipeArgs {
  TcArgs base;                 // tables, shapes, schedule, scale: the same for every layer of the launch
  LayerDesc lay[kMaxLay];
  int a_first, a_last;         // stream A: pass 1 of layers a_first..a_last (none if a_first > a_last)
  int b_first, b_last;         // stream B: pass 2 of layers b_first..b_last
  int step;                    // 1; 2 when both streams run pass 2 (the callers supplied the row statistics): stream A
                               // takes entries a_first, a_first + 2, ..., stream B entries b_first, b_first + 2, ...
  unsigned* counters;          // [kMaxLay] CTAs that have published the layer's row statistics, then [1] CTAs that are done
  unsigned target[kMaxLay];    // value a layer's counter reaches when all CTAs of this launch have published
};

// Counter sets, taken in turn by the launches (zero at load).  The last CTA of a launch to finish puts its set back to
// zero, so the set is clean for its next user 64 launches later; no memset sits between two launches.
__device__ unsigned g_layer_published[kCountSlots * kCountWords];

// One stream's resources inside the CTA.
struct StreamCtx {
  uint32_t q_smem, k_smem, bar0, tmem0;
  int n_stages;
  volatile int* abort_flag;
  volatile int* b_layer;       // CTA-wide: the layer whose pass 2 this CTA's epilogue has begun
  __device__ __forceinline__ uint32_t full_bar(int st) const { return bar0 + 8u * st; }
  __device__ __forceinline__ uint32_t empty_bar(int st) const { return bar0 + 8u * (3 + st); }
  __device__ __forceinline__ uint32_t accf_bar(int b) const { return bar0 + 8u * (6 + b); }
  // three warpgroups per stream: one barrier per (warpgroup, accumulator), so that a warpgroup sees every phase of the
  // barriers it waits on (a parity wait tells only adjacent phases apart)
  __device__ __forceinline__ uint32_t accf_bar_of(int wg, int b) const { return bar0 + 8u * (13 + 2 * wg + b); }
  __device__ __forceinline__ uint32_t acce_bar(int b) const { return bar0 + 8u * (8 + b); }
  __device__ __forceinline__ uint32_t qfull_bar() const { return bar0 + 8u * 10; }
  __device__ __forceinline__ uint32_t qempty_bar() const { return bar0 + 8u * 11; }
  __device__ __forceinline__ uint32_t drain_bar() const { return bar0 + 8u * 12; }   // used only when a wait ran out
};

// sum_e 2^(v_e * sc - m) over 32 accumulator values.  All exponentials on the special-function unit: with sixteen
// epilogue warps at 96 registers the polynomial share the single-layer kernels use made this kernel slower.
__device__ __forceinline__ float sum_ex2_32_mufu(const uint32_t (&r)[32], float sc, float m) {
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
  for (int e = 0; e < 32; e += 4) {
    s0 += ex2(fmaf(__uint_as_float(r[e]), sc, -m));
    s1 += ex2(fmaf(__uint_as_float(r[e + 1]), sc, -m));
    s2 += ex2(fmaf(__uint_as_float(r[e + 2]), sc, -m));
    s3 += ex2(fmaf(__uint_as_float(r[e + 3]), sc, -m));
  }
  return (s0 + s1) + (s2 + s3);
}
// this CTA's tiles of an entry
__device__ __forceinline__ void entry_range(const TcArgs& a, const LayerDesc& L, int& begin, int& end) {
  begin = min(L.tile_begin + (int)blockIdx.x * a.tiles_per_cta, L.tile_end);
  end = min(begin + a.tiles_per_cta, L.tile_end);
}
__device__ __forceinline__ void named_bar(int id, int n_threads = kEpiThreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n_threads) : "memory");
}

// ---- one thread: TMA loads of the stream's Q tiles and K tiles ------------------------------------------
template <bool VOTE>
__device__ __forceinline__ void producer(const StreamCtx& c, const TcArgs& a, const LayerDesc* lay, int first, int last,
                                         int step, int new_from) {
  int it = 0, run_idx = 0, st = 0;
  uint32_t st_phase = 0;
  bool ok = true;
  // Every K tile is read twice, by pass 1 and a layer later by pass 2, in the same order: pass 1 asks L2 to keep the
  // lines, pass 2 to drop them first, so that about one layer's K is live in L2 and pass 2 need not go to HBM.
  const uint64_t policy = VOTE ? l2_policy_evict_first() : l2_policy_evict_last();
  for (int j = first; j <= last && ok; j += step) {
    if (j == new_from || (j == first && j > new_from)) pdl_wait();   // inputs this launch is the first to read
    if (!VOTE) {
      // Pass 1 stays at most one layer ahead of this CTA's pass 2 (which needs the other CTAs' pass 1 of the layer
      // before, so it cannot deadlock): the two streams then share the SM to the end instead of pass 2 running on
      // alone, on half the epilogue warps, after pass 1 has raced through the list.
      const unsigned long long t0 = now_ns();
      for (unsigned spin = 1; *c.b_layer < j - kLeadEntries; ++spin) {
        if ((spin & 63u) == 0 && (*c.abort_flag || now_ns() - t0 > kWaitLimitNs)) { *c.abort_flag = 1; ok = false; break; }
        __nanosleep(100);
      }
      if (!ok) break;
    }
    const CUtensorMap* tm_q = &lay[j].tm_q;
    const CUtensorMap* tm_k = &lay[j].tm_k;
    int begin, end;
    entry_range(a, lay[j], begin, end);
    for (int pos = begin; pos < end && ok;) {
      const Run r = locate(a, pos, begin, end, false);
      ok = mbar_wait(c.qempty_bar(), (run_idx & 1) ^ 1, c.abort_flag, kPollNs);        // the run before is done with Q
      if (!ok) break;
      mbar_expect_tx(c.qfull_bar(), 2u * (uint32_t)a.R * 128u);
      const int qy = a.q_head_inner ? r.g * a.G : 0, qz = a.q_head_inner ? 0 : r.g * a.G;
      tma_load_4d(c.q_smem, tm_q, 0, qy, qz, r.s, c.qfull_bar());
      tma_load_4d(c.q_smem + kHalfBytes, tm_q, 64, qy, qz, r.s, c.qfull_bar());
      int tok = a.tab.cu_at(r.s) + r.t0 * kTileKeys;
      for (int i = 0; i < r.count; ++i, ++it, tok += kTileKeys) {
        ok = mbar_wait(c.empty_bar(st), st_phase ^ 1u, c.abort_flag, kPollNs);
        if (!ok) break;
        const uint32_t fb = c.full_bar(st), dst = c.k_smem + (uint32_t)st * kStageBytes;
        mbar_expect_tx(fb, kStageBytes);
        const int ky = a.k_head_inner ? r.g : tok, kz = a.k_head_inner ? tok : r.g;
        tma_load_3d_hint(dst, tm_k, 0, ky, kz, fb, policy);
        tma_load_3d_hint(dst + kHalfBytes, tm_k, 64, ky, kz, fb, policy);
        if (++st == c.n_stages) { st = 0; st_phase ^= 1u; }
      }
      pos += r.count;
      ++run_idx;
    }
  }
  if (!ok) {
    // give loads already in flight a bounded chance to land before the CTA's shared memory goes away
    const unsigned long long t0 = now_ns();
    for (int s2 = 0; s2 < c.n_stages; ++s2) {
      const int last_it = it - 1 - ((it - 1 - s2) % c.n_stages + c.n_stages) % c.n_stages;   // last issue into stage s2
      if (it == 0 || last_it < 0) continue;
      while (!mbar_try(c.full_bar(s2), (last_it / c.n_stages) & 1) && now_ns() - t0 < kWaitLimitNs) {}
    }
  }
}

// ---- one thread: the stream's MMAs, one 128 x 128 x 128 product per tile into one of two accumulators --------
template <bool VOTE, int NWG = 2>
__device__ __forceinline__ void issuer(const StreamCtx& c, const TcArgs& a, const LayerDesc* lay, int first, int last,
                                       int step) {
  // pass 1: D[row, key] = Q K^T (A = Q, B = K); pass 2: D[key, row] = K Q^T (A = K, B = Q, N = R)
  const uint32_t idesc = VOTE ? instr_desc(kTileKeys, a.R) : instr_desc(128, kTileKeys);
  const uint64_t q_desc0 = smem_desc(c.q_smem), k_desc0 = smem_desc(c.k_smem);
  const uint64_t hi = (uint64_t)(kHalfBytes >> 4);
  int it = 0, run_idx = 0, st = 0, b = 0;
  uint32_t st_phase = 0, b_phase = 0;
  uint64_t k_desc = k_desc0;
  bool ok = true;
  for (int j = first; j <= last && ok; j += step) {
  int begin, end;
  entry_range(a, lay[j], begin, end);
  for (int pos = begin; pos < end && ok;) {
    const Run r = locate(a, pos, begin, end, false);
    ok = mbar_wait(c.qfull_bar(), run_idx & 1, c.abort_flag, kPollNs);
    if (!ok) break;
    for (int i = 0; i < r.count; ++i, ++it) {
      ok = mbar_wait(c.full_bar(st), st_phase, c.abort_flag, kPollNs) && mbar_wait(c.acce_bar(b), b_phase ^ 1u, c.abort_flag, kPollNs);
      if (!ok) break;
      tc_fence_after();
      const uint32_t d0 = c.tmem0 + (uint32_t)(b * 128);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const uint64_t off = (uint64_t)((ks & 3) * 2) + (ks >> 2) * hi;
        if (VOTE) tc_mma(d0, k_desc + off, q_desc0 + off, idesc, ks > 0);
        else tc_mma(d0, q_desc0 + off, k_desc + off, idesc, ks > 0);
      }
      tc_commit(c.empty_bar(st));       // K stage free once these MMAs have read it
      tc_commit(NWG == 2 ? c.accf_bar(b) : c.accf_bar_of(it % NWG, b));   // accumulator ready for the epilogue
      k_desc += (uint64_t)(kStageBytes >> 4);
      if (++st == c.n_stages) { st = 0; st_phase ^= 1u; k_desc = k_desc0; }
      if (++b == 2) { b = 0; b_phase ^= 1u; }
    }
    tc_commit(c.qempty_bar());          // Q tile free once the run's MMAs are done
    pos += r.count;
    ++run_idx;
  }
  }
  if (!ok) {
    // gave up: the MMAs this thread has issued must be through before the accumulators are released
    tc_commit(c.drain_bar());
    const unsigned long long t0 = now_ns();
    while (!mbar_try(c.drain_bar(), 0) && now_ns() - t0 < kWaitLimitNs) {}
  }
}

// ---- 256 threads: pass 1, row statistics (stream A) ----------------------------------------------------------
__device__ __forceinline__ void epilogue_rows(const StreamCtx& c, const TcArgs& a, const PipeArgs& pa, int et, int warp,
                                              float* stat_m, float* stat_z) {
  const int wg = et >> 7, row = et & 127, lane = et & 31;
  const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
  const float sc = a.scale_log2;
  const int R = a.R;
  int it = 0;
  bool ok = true;
  for (int j = pa.a_first; j <= pa.a_last; ++j) {
  const LayerDesc& L = pa.lay[j];
  int begin, end;
  entry_range(a, L, begin, end);
  for (int pos = begin; pos < end;) {
    const Run r = locate(a, pos, begin, end, false);
    const int seg = r.s * a.n_kv_heads + r.g;
    const int first_cta = (r.seg_tile0 - L.tile_begin) / a.tiles_per_cta;
    float m = 0.f, z = 0.f;                                   // fixed reference 0 on the fast path
    for (int i = 0; i < r.count; ++i, ++it) {
      if ((it & 1) != wg) continue;
      const int b = it & 1;
      if (ok) ok = mbar_wait(c.accf_bar(b), (it >> 1) & 1, c.abort_flag, kPollNs);
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
        if (nv <= 0) return;                                   // wholly past the segment's end
        if (nv >= 32) {
          const float zc = sum_ex2_32_mufu(rr, sc, m);
          const float zn = z + zc;
          if (zn < INFINITY && zn > kTinySum) { z = zn; return; }
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
      L.part_m[((long long)seg * a.slot_stride + slot) * R + row] = M;
      L.part_z[((long long)seg * a.slot_stride + slot) * R + row] = Z;
    }
    named_bar(1);
    pos += r.count;
  }
  // This CTA's row statistics of layer j are written (the barrier above orders the other threads' stores before
  // this thread's release): one more CTA has published.
  if (et == 0 && ok) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(pa.counters + j) : "memory");
  if (et == 0 && j < 24) trace_mark(a.trace, 8 + 2 * j);
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
    s3 += ex2(fmaf(__uint_as_float(r[e + 3]), sc, -l4.w));
  }
  return (s0 + s1) + (s2 + s3);
}

// sum_e 2^(v_e * sc - lse_e) over 16 accumulator values
__device__ __forceinline__ float vote_chunk16(const uint32_t (&r)[16], float sc, const float* lse) {
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
  for (int e = 0; e < 16; e += 4) {
    const float4 l4 = *reinterpret_cast<const float4*>(lse + e);
    s0 += ex2(fmaf(__uint_as_float(r[e]), sc, -l4.x));
    s1 += ex2(fmaf(__uint_as_float(r[e + 1]), sc, -l4.y));
    s2 += ex2(fmaf(__uint_as_float(r[e + 2]), sc, -l4.z));
    s3 += ex2(fmaf(__uint_as_float(r[e + 3]), sc, -l4.w));
  }
  return (s0 + s1) + (s2 + s3);
}

// ---- 256 threads: pass 2, votes (stream B) ---------------------------------------------------------------------
// `first`, `last`, pa.step: the entries this stream takes; `bar_id`: the named barrier of its 256 threads; `is_b`: the
// stream pass 1 of the same CTA keeps its distance to.
template <int NWG>
__device__ __forceinline__ void epilogue_votes(const StreamCtx& c, const TcArgs& a, const PipeArgs& pa, int et, int warp,
                                               float* lse2, int first, int last, int bar_id, bool is_b) {
  const int wg = et >> 7, row = et & 127, lane = et & 31;
  const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
  const float sc = a.scale_log2;
  const float inv_g = 1.0f / (float)a.G;
  const int R = a.R;
  int it = 0, run_idx = 0;
  int own0 = 0, own1 = 0;               // this warpgroup's tiles so far on either accumulator (three warpgroups)
  bool ok = true;
  for (int j = first; j <= last; j += pa.step) {
  const LayerDesc& L = pa.lay[j];
  if (pa.step == 1 && j >= pa.a_first && j <= pa.a_last && !L.lse.lse_opt) {
    // the layer's pass 1 is part of this launch: wait until every CTA has published its row statistics (all CTAs
    // are resident, and stream A waits for nothing, so the count gets there; bounded all the same)
    if (et == 0 && ok) {
      const unsigned long long t0 = now_ns();
      for (unsigned spin = 1;; ++spin) {
        unsigned v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(pa.counters + j) : "memory");
        if ((int)(v - pa.target[j]) >= 0) break;
        if ((spin & 63u) == 0 && (*c.abort_flag || now_ns() - t0 > kWaitLimitNs)) { *c.abort_flag = 1; break; }
        __nanosleep(64);
      }
    }
    named_bar(bar_id, NWG * 128);
    ok = ok && *c.abort_flag == 0;
  }
  if (et == 0 && is_b) *c.b_layer = j;
  if (et == 0 && is_b && j < 24) trace_mark(a.trace, 9 + 2 * j);
  int begin, end;
  entry_range(a, L, begin, end);
  for (int pos = begin; pos < end;) {
    const Run r = locate(a, pos, begin, end, false);
    const int seg = r.s * a.n_kv_heads + r.g;
    const int first_cta = (r.seg_tile0 - L.tile_begin) / a.tiles_per_cta;
    float* lse = lse2 + 128 * (run_idx & 1);
    {
      // the rows' log-sum-exp (log2 units): the caller's, or the per-CTA partials of this segment merged (two
      // neighbouring lanes share a row)
      const int n_slots = (r.seg_tile0 - L.tile_begin + r.tiles_seg - 1) / a.tiles_per_cta - first_cta + 1;
      const int rr = (et >> 1) < R ? (et >> 1) : -1;
      const int half = et & 1;
      float l2;
      if (L.lse.lse_opt) {
        l2 = rr >= 0 ? L.lse.caller_lse(r.s, r.g, rr, a.G, a.window, a.q_head_inner != 0) : 0.f;
      } else {
        const bool has_win = L.lse.win_m != nullptr && rr >= 0;
        l2 = merged_row_lse(L.part_m + (long long)seg * a.slot_stride * R, L.part_z + (long long)seg * a.slot_stride * R,
                            n_slots, R, rr, half, 2, has_win, has_win ? L.lse.win_m[(long long)seg * R + rr] : 0.f,
                            has_win ? L.lse.win_z[(long long)seg * R + rr] : 0.f);
      }
      if (half == 0 && rr >= 0) lse[rr] = l2;
    }
    named_bar(bar_id, NWG * 128);
    if (et == 0 && is_b && run_idx == 0) trace_mark(a.trace, 3);
    for (int i = 0; i < r.count; ++i, ++it) {
      const int b = it & 1;
      if (NWG == 2) {
        if ((it & 1) != wg) continue;
        if (ok) ok = mbar_wait(c.accf_bar(b), (it >> 1) & 1, c.abort_flag, kPollNs);
      } else {
        if (it % NWG != wg) continue;
        const int mine = b ? own1++ : own0++;
        if (ok) ok = mbar_wait(c.accf_bar_of(wg, b), mine & 1, c.abort_flag, kPollNs);
      }
      ok = __all_sync(0xffffffffu, ok) != 0;
      if (!ok) continue;
      tc_fence_after();
      const int key0 = (r.t0 + i) * kTileKeys;
      const uint32_t tb = c.tmem0 + lane_sel + (uint32_t)(b * 128);
      float acc = 0.f;
      auto release = [&]() {
        // the accumulator is in registers: hand its TMEM buffer back before the arithmetic and the vote's store
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(c.acce_bar(b));
      };
      if (NWG == 2) {
        uint32_t ra[32], rb[32];
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
      } else {
        // three warpgroups per stream share the register file: rounds of 16 columns (R is a multiple of 32)
        uint32_t ra[16], rb[16];
        tc_ld16_issue(tb, ra);
#pragma unroll 1
        for (int c0 = 0; c0 < R; c0 += 32) {
          tc_ld_wait16(ra);
          tc_ld16_issue(tb + c0 + 16, rb);
          acc += vote_chunk16(ra, sc, lse + c0);
          tc_ld_wait16(rb);
          if (c0 + 32 < R) tc_ld16_issue(tb + c0 + 32, ra); else release();
          acc += vote_chunk16(rb, sc, lse + c0 + 16);
        }
      }
      const int jk = key0 + row;
      if (jk < r.n_hist) L.vote[a.tab.hist_at(r.s) * a.n_kv_heads + (long long)r.g * r.n_hist + jk] = acc * inv_g;
    }
    pos += r.count;
    ++run_idx;
  }
  }
}

// DUAL: both streams run pass 2 (every layer of the list came with its row statistics), each on every other entry.
template <bool DUAL>
__global__ void __launch_bounds__(DUAL ? kDualThreads : kPipeThreads, 1)
k_score_pipe(const __grid_constant__ PipeArgs pa) {
  // Shared memory, all dynamic and 1024-byte aligned (the swizzled tiles need it):
  //   [Q of A 32 KB][Q of B 32 KB][K ring of A 2 x 32 KB][K ring of B 3 x 32 KB][mbarriers, flags 512 B]
  //   [stat_m, stat_z of A 1 KB][log-sum-exp rows of B 2 x 512 B]
  extern __shared__ __align__(1024) unsigned char smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  unsigned char* tail = smem + 2 * kQBytes + (kStagesA + kStagesB) * kStageBytes;
  uint32_t& tmem_base_sh = *reinterpret_cast<uint32_t*>(tail + 2 * kBarBytesPerStream);
  int& abort_sh = *reinterpret_cast<int*>(tail + 2 * kBarBytesPerStream + 4);
  int& b_layer_sh = *reinterpret_cast<int*>(tail + 2 * kBarBytesPerStream + 8);   // the layer stream B's epilogue has begun
  float* stat_m = reinterpret_cast<float*>(tail + 512);
  float* stat_z = stat_m + 128;
  float* lse2 = stat_m + 256;
  const TcArgs& a = pa.base;
  const bool has_a = pa.a_first <= pa.a_last, has_b = pa.b_first <= pa.b_last;
  const int lay_lo = has_b ? min(pa.b_first, has_a ? pa.a_first : pa.b_first) : pa.a_first;
  const int lay_hi = has_a ? max(pa.a_last, has_b ? pa.b_last : pa.a_last) : pa.b_last;
  if ((smem_u32(smem) & 1023u) != 0) {                      // never run on a skewed layout (uniform over the CTA)
    if (tid == 0)
      for (int j = lay_lo; j <= lay_hi; ++j)
        if (pa.lay[j].status) atomicExch(pa.lay[j].status, (int)SLKV_ERR_BAD_ALIGN);
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
  ca.b_layer = cb.b_layer = &b_layer_sh;

  if (tid == 0) trace_mark(a.trace, 0);
  if (tid == 0 && a.trace) a.trace[(size_t)blockIdx.x * kTraceSlots + 60] = (unsigned long long)clock64();
  if (tid == 0) {
    if (has_a) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&pa.lay[pa.a_first].tm_k)) : "memory");
    if (has_b) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&pa.lay[pa.b_first].tm_k)) : "memory");
    if (has_a) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&pa.lay[pa.a_first].tm_q)) : "memory");
    if (has_b) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&pa.lay[pa.b_first].tm_q)) : "memory");
    abort_sh = 0;
    b_layer_sh = has_b ? pa.b_first - 1 : 1 << 30;
    for (int s = 0; s < 2; ++s) {
      const StreamCtx& c = s ? cb : ca;
      for (int st = 0; st < 3; ++st) { mbar_init(c.full_bar(st), 1); mbar_init(c.empty_bar(st), 1); }
      for (int b = 0; b < 2; ++b) { mbar_init(c.accf_bar(b), 1); mbar_init(c.acce_bar(b), 4); }
      for (int g = 0; g < 6; ++g) mbar_init(c.accf_bar_of(g >> 1, g & 1), 1);
      mbar_init(c.qfull_bar(), 1);
      mbar_init(c.qempty_bar(), 1);
      mbar_init(c.drain_bar(), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // rows of a Q tile beyond R are never written by TMA: keep them zero
  if (a.R != 128) {
    for (int i = tid; i < 2 * kQBytes / 16; i += (int)blockDim.x) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
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
  // With both streams on the vote pass the launch behind this one is another of its kind, and none of its CTAs fits
  // on an SM this launch holds: released now they would only sit on the SMs left to the selection kernels until this
  // launch ends.  They are released when this CTA is done instead.
  if (!DUAL) pdl_launch_dependents();

  // Stream A reads its layers' Q and K for the first time and overwrites row statistics an earlier launch may still
  // be merging: all its roles wait for the work before this launch.  Stream B's loads and MMAs need only Q and K,
  // which are inputs, and for the pending layer have been read by the launch before: they start at once; its
  // epilogue needs that launch's row statistics and waits.
  if (warp == 0) {
    if (lane == 0 && has_a) {
      if (DUAL) producer<true>(ca, a, pa.lay, pa.a_first, pa.a_last, pa.step, pa.a_first);
      else producer<false>(ca, a, pa.lay, pa.a_first, pa.a_last, 1, pa.a_first);
    }
  } else if (warp == 1) {
    if (lane == 0 && has_a) {
      if (DUAL) issuer<true, kDualWgs>(ca, a, pa.lay, pa.a_first, pa.a_last, pa.step);
      else issuer<false>(ca, a, pa.lay, pa.a_first, pa.a_last, 1);
    }
  } else if (warp == 2) {
    // normally entry 0 was read by the launch before; with both streams on pass 2 every entry is new to this launch
    if (lane == 0 && has_b) producer<true>(cb, a, pa.lay, pa.b_first, pa.b_last, pa.step, DUAL ? pa.b_first : 1);
  } else if (warp == 3) {
    if (lane == 0 && has_b) { if (DUAL) issuer<true, kDualWgs>(cb, a, pa.lay, pa.b_first, pa.b_last, pa.step); else issuer<true>(cb, a, pa.lay, pa.b_first, pa.b_last, pa.step); }
  } else if (warp < (DUAL ? 4 + 4 * kDualWgs : 12)) {
    if (has_a) {
      pdl_wait();
      if (tid == 128) trace_mark(a.trace, 1);
      if (DUAL) epilogue_votes<kDualWgs>(ca, a, pa, tid - 128, warp, stat_m, pa.a_first, pa.a_last, 1, false);
      else epilogue_rows(ca, a, pa, tid - 128, warp, stat_m, stat_z);
      if (tid == 128) trace_mark(a.trace, 5);
    }
  } else {
    if (has_b) {
      pdl_wait();
      constexpr int kFirstB = DUAL ? 128 + 128 * kDualWgs : 384;
      if (tid == kFirstB) trace_mark(a.trace, 7);
      if (DUAL) epilogue_votes<kDualWgs>(cb, a, pa, tid - kFirstB, warp, lse2, pa.b_first, pa.b_last, 2, true);
      else epilogue_votes<2>(cb, a, pa, tid - kFirstB, warp, lse2, pa.b_first, pa.b_last, 2, true);
      if (tid == kFirstB) trace_mark(a.trace, 6);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (DUAL) pdl_launch_dependents();
  if (abort_sh && tid == 0)
    for (int j = lay_lo; j <= lay_hi; ++j)
      if (pa.lay[j].status) atomicExch(pa.lay[j].status, (int)SLKV_ERR_DEVICE_TIMEOUT);
  if (tid == 0) trace_mark(a.trace, 4);
  if (tid == 0 && a.trace) a.trace[(size_t)blockIdx.x * kTraceSlots + 61] = (unsigned long long)clock64();
  if (tid == 0) {
    // every thread of this CTA is past its last use of the counters (the barrier above)
    unsigned prev;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(prev) : "l"(pa.counters + kMaxLay) : "memory");
    if (prev == gridDim.x - 1) {
      for (int j = 0; j <= kMaxLay; ++j) pa.counters[j] = 0;
      __threadfence();
    }
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace

bool score_pipe_supported(const Problem& pb) {
  return tensor_path_supported(pb.p) && pb.R <= 128;
}

// One launch: pass 1 of plans a[0..n_a) beside pass 2 of `pending` (the layer whose pass 1 an earlier launch did;
// may be null) and of a[0..n_a-1), or of all of a[] when `finish` is set.  The plans share one shape and schedule.
cudaError_t launch_score_pipe(const TcPlan* pending, const TcPlan* const* a, int n_a, bool finish, bool votes_only,
                              cudaStream_t st, int* launches) {
  if (n_a > kPipeMaxLayers) return cudaErrorInvalidValue;
  if (votes_only && pending) return cudaErrorInvalidValue;     // nothing stays pending between vote-only launches
  // Without cooperative launches (refused once on this device) no launch may hold both passes of a layer: one layer's
  // pass 1 per launch, beside pass 2 of the layer before.
  static thread_local bool no_coop[64] = {};
  static const bool env_no_coop = [] {                // SLKV_NO_COOPERATIVE=1: behave as if they were refused (tests)
    const char* v = std::getenv("SLKV_NO_COOPERATIVE");
    return v && v[0] == '1';
  }();
  {
    int d = 0;
    if (env_no_coop && cudaGetDevice(&d) == cudaSuccess && d >= 0 && d < 64) no_coop[d] = true;
    if (!votes_only && cudaGetDevice(&d) == cudaSuccess && d >= 0 && d < 64 && no_coop[d] &&
        (n_a > 1 || (n_a == 1 && finish))) {
      const TcPlan* prev = pending;
      for (int i = 0; i < n_a; ++i) {
        cudaError_t e1 = launch_score_pipe(prev, a + i, 1, false, false, st, launches);
        if (e1 != cudaSuccess) return e1;
        prev = a[i];
      }
      return finish ? launch_score_pipe(prev, nullptr, 0, true, false, st, launches) : cudaSuccess;
    }
  }
  const TcPlan* any = pending && pending->n_cta > 0 ? pending : nullptr;
  for (int i = 0; i < n_a && !any; ++i)
    if (a[i]->n_cta > 0) any = a[i];
  if (!any) return cudaSuccess;                       // no history anywhere: nothing to score
  static thread_local int configured_dev = -1;
  static thread_local unsigned* counters_base = nullptr;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (configured_dev != dev) {
    e = cudaFuncSetAttribute(k_score_pipe<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPipeSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_score_pipe<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPipeSmem);
    if (e != cudaSuccess) return e;
    void* sym = nullptr;
    e = cudaGetSymbolAddress(&sym, g_layer_published);
    if (e != cudaSuccess) return e;
    counters_base = static_cast<unsigned*>(sym);
    configured_dev = dev;
  }
  PipeArgs pa;
  std::memset(&pa, 0, sizeof(pa));
  pa.base = any->a;
  pa.base.part_m = pa.base.part_z = pa.base.vote = nullptr;
  pa.base.status = nullptr;
  // A layer goes in as one entry, or as two (its first and second half of the segments) when the halves are whole
  // segments and equal: pass 2 of an entry then follows its pass 1 after half a layer's time and half a layer's K.
  const TcArgs& sh = any->a;
  const int total = sh.total_tiles;
  int groups = 1;
  if (kMaxGroups >= 2 && total % 2 == 0 && sh.tab.n_inline > 0) {
    const int mid = total / 2;
    for (int q = 0; q < sh.tab.n_inline && groups == 1; ++q) {
      const int t_seq = sh.tab.tile_off[q + 1] - sh.tab.tile_off[q];
      for (int g = 0; g < sh.n_kv_heads; ++g)
        if (sh.n_kv_heads * sh.tab.tile_off[q] + g * t_seq == mid) { groups = 2; break; }
    }
  }
  int n_cta = any->n_cta;
  if (groups == 2) {
    const int per_group = total / 2;
    int tpc = (per_group + n_cta - 1) / n_cta;
    pa.base.tiles_per_cta = tpc;
    n_cta = (per_group + tpc - 1) / tpc;
  }
  auto fill = [&](int j, const TcPlan* p, int group) {
    pa.lay[j].tm_q = p->tm_q; pa.lay[j].tm_k = p->tm_k;
    pa.lay[j].part_m = p->a.part_m; pa.lay[j].part_z = p->a.part_z; pa.lay[j].vote = p->a.vote;
    pa.lay[j].status = p->a.status;
    pa.lay[j].lse = p->a.lse;
    pa.lay[j].tile_begin = groups == 2 ? group * (total / 2) : 0;
    pa.lay[j].tile_end = groups == 2 ? (group + 1) * (total / 2) : total;
  };
  const bool has_pending = pending && pending->n_cta > 0;
  if (has_pending) fill(0, pending, groups - 1);      // what is pending of a layer is its last group
  int n_live = 0;
  for (int i = 0; i < n_a; ++i)
    if (a[i]->n_cta > 0)
      for (int g = 0; g < groups; ++g) fill(++n_live, a[i], g);     // layers without history take no part
  pa.a_first = 1; pa.a_last = n_live;
  pa.b_first = has_pending ? 0 : 1;
  pa.b_last = finish ? n_live : n_live - 1;
  pa.step = 1;
  if (votes_only) {                                   // both streams on pass 2, every other entry each
    pa.step = 2;
    pa.b_first = 2;
    pa.b_last = n_live;
  }
  if (pa.a_first > pa.a_last && pa.b_first > pa.b_last) return cudaSuccess;
  pa.base.trace = tensor_trace_buffer(0, n_cta);
  // counters of this launch: a slot of the table, zeroed on the stream before the kernel
  static std::atomic<unsigned> launch_seq{0};
  pa.counters = counters_base + (size_t)(launch_seq.fetch_add(1) % kCountSlots) * kCountWords;
  const bool waits_inside = !votes_only && pa.b_last >= pa.a_first && pa.a_last >= pa.a_first;   // a layer's two passes in one launch
  const unsigned extra = waits_inside && take_expire_next_wait() ? 1u : 0u;       // diagnostics: a wait that runs out
  for (int j = 0; j < kMaxLay; ++j) pa.target[j] = (unsigned)n_cta + extra;
  // CTAs that wait for one another must all be resident: cooperative launch.  Dependent launch on top where the
  // device takes both (the kernel waits for the launch before it exactly where it needs that launch's results).
  static thread_local int pdl_with_coop[64] = {};     // per device: 0 untried, 1 works, -1 refused
  int& pc = pdl_with_coop[dev < 64 ? dev : 0];
  for (int attempt = 0; attempt < 2; ++attempt) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_cta);
    cfg.blockDim = dim3(votes_only ? kDualThreads : kPipeThreads);
    cfg.dynamicSmemBytes = kPipeSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[3];
    int n = 0;
    {
      // ahead of the selections and gathers that become ready at the same moment on the side streams: when SMs
      // come free, this kernel's CTAs are placed first
      int least = 0, greatest = 0;
      if (cudaDeviceGetStreamPriorityRange(&least, &greatest) == cudaSuccess && greatest != least) {
        attr[n].id = cudaLaunchAttributePriority;
        attr[n].val.priority = greatest;
        ++n;
      }
    }
    if (waits_inside) {
      attr[n].id = cudaLaunchAttributeCooperative;
      attr[n].val.cooperative = 1;
      ++n;
    }
    const bool with_pdl = !waits_inside || pc >= 0;
    if (with_pdl) {
      attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[n].val.programmaticStreamSerializationAllowed = 1;
      ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    cudaError_t le;
    {
      LaunchScope scope(KID_SCORE_PIPE, st, launches);
      le = votes_only ? cudaLaunchKernelEx(&cfg, k_score_pipe<true>, pa) : cudaLaunchKernelEx(&cfg, k_score_pipe<false>, pa);
    }
    if (le == cudaSuccess) {
      if (waits_inside && with_pdl) pc = 1;
      return cudaSuccess;
    }
    if (!waits_inside) return le;
    (void)cudaGetLastError();                         // not a sticky error: the launch was refused
    --*launches;
    if (with_pdl && pc != 1) { pc = -1; continue; }   // once more without dependent launch
    // cooperative launches do not work here: the list goes out one layer per launch from now on
    no_coop[dev < 64 ? dev : 0] = true;
    return launch_score_pipe(pending, a, n_a, finish, votes_only, st, launches);
  }
  return cudaErrorLaunchFailure;
}

// The most layers one launch takes (pass 1); callers that queue layers launch when they have this many.
int score_pipe_max_layers() { return kPipeMaxLayers; }

}  // namespace slkv
