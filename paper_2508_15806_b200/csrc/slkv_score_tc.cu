// Window relevance scores on the 5th-generation tensor cores (Sec. 3.4, Eq. 7; Algorithm 3 l.6; Eq. 3-4).
//
// bf16, head_dim 128.  Two persistent kernels share one schedule: the history keys of all (sequence,
// KV head) segments form one list of 128-key tiles, split evenly over one CTA per SM.
//   pass 1 (row statistics)  S = Q K^T per tile with the G*w query rows as the M dimension, so that a
//           TMEM lane -- one thread -- owns a query row: running max and sum of 2^(s - max) stay in
//           registers; per CTA and segment one (max, sum) pair per row goes to global memory.
//   pass 2 (votes)           S^T = K Q^T per tile with the keys as the M dimension, so that a thread owns
//           a key: vote[j] = (1/G) sum_rows 2^(s_rj - lse_r) is a thread-local sum and a coalesced store.
// Warp roles: warp 0 issues TMA loads (128-byte-swizzled K-major tiles, no multicast), warps 1 and 2 issue
// tcgen05.mma (alternate tiles) into TMEM accumulators and commit to mbarriers, warps 4..11 (two warpgroups, alternating
// tiles) read TMEM with tcgen05.ld and do the softmax arithmetic in fp32.
// Every mbarrier wait is bounded by a wall-clock limit; when one runs out the CTA raises
// SLKV_ERR_DEVICE_TIMEOUT in the status word, stops waiting everywhere, releases TMEM and returns.
#include <cuda.h>

#include <atomic>

#include "slkv_internal.cuh"
#include "slkv_tc_device.cuh"

namespace slkv {
namespace {

// Grid-wide barrier of the fused kernel (both passes in one launch): one arrival counter per launch, taken in
// turn from a small table in the module's globals (zero at load).  atom.inc wraps the counter back to zero with
// the last arrival, so a waiter -- which has arrived itself, hence has seen the counter above zero -- is done
// when it reads zero.  Beside it sits an exit counter: the last CTA to leave the kernel puts both words back to zero,
// so a launch whose wait ran out (some CTAs never arrived, the arrival counter did not wrap) still leaves the slot
// clean for its next user 64 launches later.  The kernel is launched cooperatively (all CTAs resident); the wait is
// bounded all the same.
constexpr int kBarrierSlots = 64;
__device__ unsigned g_grid_arrivals[2 * kBarrierSlots];

__device__ __forceinline__ bool grid_barrier(unsigned* counter, unsigned n_arrivals, volatile int* abort_flag) {
  // Called by one thread after a CTA-wide barrier: the release on the arrival makes the CTA's earlier writes
  // visible to whoever acquires the counter afterwards.  n_arrivals = the grid size (a diagnostic launch asks for
  // one more than will ever come, so that the wait runs out).
  unsigned prev;
  asm volatile("atom.acq_rel.gpu.global.inc.u32 %0, [%1], %2;" : "=r"(prev) : "l"(counter), "r"(n_arrivals - 1) : "memory");
  if (prev == n_arrivals - 1) return true;
  const unsigned long long t0 = now_ns();
  for (unsigned it = 1;; ++it) {
    unsigned c;
    asm volatile("ld.acquire.gpu.u32 %0, [%1];" : "=r"(c) : "l"(counter) : "memory");
    if (c == 0) return true;
    if ((it & 15u) == 0) {
      if (*abort_flag) return false;
      if (now_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
    }
    __nanosleep(32);
  }
}

// MODE 1: row statistics pass only; MODE 2: vote pass only; MODE 3: both, separated by a grid-wide barrier.
template <int MODE>
__global__ void __launch_bounds__(kThreads, 1)
k_score_tc(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ TcArgs a) {
  // Shared memory, all dynamic and 1024-byte aligned (the swizzled tiles need it):
  //   [Q tile: MT x 32 KB][K ring: n_stages x 32 KB][mbarriers, flags: 512 B][row statistics: 2 KB]
  extern __shared__ __align__(1024) unsigned char smem[];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int MT = a.MT, R = a.R, kStages = a.n_stages;
  const int buf_cols = MT * 128;
  const int n_bufs = 512 / buf_cols;                        // 4 or 2 TMEM accumulator buffers
  const int q_half_bytes = MT * 128 * 128;                  // one 64-element half of the (padded) Q tile

  unsigned char* tail = smem + 2 * q_half_bytes + kStages * kStageBytes;
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(tail);
  uint32_t& tmem_base_sh = *reinterpret_cast<uint32_t*>(tail + 256);
  int& abort_sh = *reinterpret_cast<int*>(tail + 260);
  float* stats = reinterpret_cast<float*>(tail + 512);      // pass 1: stat_m[256], stat_z[256]; pass 2: lse[2][256]
  float* stat_m = stats;
  float* stat_z = stats + 256;
  if ((smem_u32(smem) & 1023u) != 0) {                      // never run on a skewed layout (uniform over the CTA)
    if (tid == 0 && a.status) atomicExch(a.status, (int)SLKV_ERR_BAD_ALIGN);
    return;
  }
  const uint32_t q_smem = smem_u32(smem);
  const uint32_t k_smem = q_smem + 2 * q_half_bytes;
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int st) { return bar0 + 8u * st; };
  auto empty_bar = [&](int st) { return bar0 + 8u * (kStages + st); };
  auto accf_bar = [&](int b) { return bar0 + 8u * (2 * kStages + b); };
  auto acce_bar = [&](int b) { return bar0 + 8u * (2 * kStages + 4 + b); };
  const uint32_t qfull_bar = bar0 + 8u * (2 * kStages + 8), qempty_bar = qfull_bar + 8u;
  auto drain_bar = [&](int issuer) { return bar0 + 8u * (2 * kStages + 10 + issuer); };    // used only when a wait ran out
  volatile int* abort_flag = &abort_sh;

  const int begin = blockIdx.x * a.tiles_per_cta;
  const int end = min(begin + a.tiles_per_cta, a.total_tiles);

  if (tid == 0) trace_mark(a.trace, 0);
  if (tid == 0) {
    // the tensor maps travel as kernel parameters: have them fetched while the CTA sets itself up
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_k)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_q)) : "memory");
    abort_sh = 0;
    for (int st = 0; st < kStages; ++st) { mbar_init(full_bar(st), 1); mbar_init(empty_bar(st), 1); }
    for (int b = 0; b < 4; ++b) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), 4); }
    mbar_init(qfull_bar, 1);
    mbar_init(qempty_bar, 2);                                 // one arrival per MMA issuer
    mbar_init(drain_bar(0), 1);
    mbar_init(drain_bar(1), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // rows of the Q tile beyond R are never written by TMA: keep them zero
  if (R != MT * 128) {
    for (int i = tid; i < 2 * q_half_bytes / 16; i += kThreads) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
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
  // Everything above touched only this CTA's own resources.  Pass 1 reads its inputs after the kernels
  // before it have finished.  In pass 2 the loads and the tensor-core work need only Q and K, which pass 1
  // has already read, so they start at once; the epilogue alone waits for pass 1's row statistics.
  constexpr int kFirstPass = MODE == 2 ? 2 : 1, kLastPass = MODE == 1 ? 1 : 2;
  pdl_launch_dependents();
  if (MODE != 2 && warp >= 4) {
    bool ragged = false;                                            // a segment's ragged last tile in this CTA's range?
    for (int pos = begin; pos < end;) {
      const Run r = locate(a, pos, begin, end, false);
      ragged |= r.t0 + r.count == r.tiles_seg && (r.n_hist & (kTileKeys - 1)) != 0;
      pos += r.count;
    }
    if (ragged) {                                                   // instruction-cache warm-up, results unused
      float mw = 0.f, zw = 0.f;
      tile_row_stats_exact(tmem_base + ((uint32_t)((warp & 3) * 32) << 16), 0.f, kTileKeys - 1, mw, zw);
      if (zw == 12345.f) abort_sh = 0;                              // keeps the call alive; writes what is there
    }
  }
  if (MODE != 2 || warp >= 4 || a.fresh_inputs) pdl_wait();
  if (tid == 0) trace_mark(a.trace, 1);

  // pass 2 walks the CTA's tiles backwards: the last ones read are likeliest in L2
  auto first_pos = [&](bool REV) { return REV ? end - 1 : begin; };
  auto more = [&](int pos, bool REV) { return REV ? pos >= begin : pos < end; };
  auto advance = [&](int pos, const Run& r, bool REV) { return REV ? pos - r.count : pos + r.count; };
  auto tile_of = [&](const Run& r, int i, bool REV) { return r.t0 + (REV ? r.count - 1 - i : i); };

  // The two single-thread loops below are the pipeline's metronome: whatever they spend per tile between two
  // issues is dead time for the tensor pipe (a tcgen05.mma issue blocks its thread while the pipe is busy),
  // so ring positions and phase bits advance by increments (no divisions) and the operand descriptors are
  // built once.
  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int it = 0, run_idx = 0, st = 0;
      uint32_t st_phase = 0;                                             // parity of the ring pass in progress
      bool ok = true;
     for (int pass = kFirstPass; pass <= kLastPass && ok; ++pass) {
      const bool REV = pass == 2;
      for (int pos = first_pos(REV); more(pos, REV) && ok;) {
        const Run r = locate(a, pos, begin, end, REV);
        ok = mbar_wait(qempty_bar, (run_idx & 1) ^ 1, abort_flag);      // previous run's MMAs are done with Q
        if (!ok) break;
        mbar_expect_tx(qfull_bar, 2u * (uint32_t)R * 128u);
        const int qy = a.q_head_inner ? r.g * a.G : 0, qz = a.q_head_inner ? 0 : r.g * a.G;
        tma_load_4d(q_smem, &tm_q, 0, qy, qz, r.s, qfull_bar);
        tma_load_4d(q_smem + q_half_bytes, &tm_q, 64, qy, qz, r.s, qfull_bar);
        int tok = a.tab.cu_at(r.s) + tile_of(r, 0, REV) * kTileKeys;
        const int tok_step = REV ? -kTileKeys : kTileKeys;
        for (int i = 0; i < r.count; ++i, ++it, tok += tok_step) {
          ok = mbar_wait(empty_bar(st), st_phase ^ 1u, abort_flag);
          if (!ok) break;
          const uint32_t fb = full_bar(st), dst = k_smem + (uint32_t)st * kStageBytes;
          mbar_expect_tx(fb, kStageBytes);
          const int ky = a.k_head_inner ? r.g : tok, kz = a.k_head_inner ? tok : r.g;
          tma_load_3d(dst, &tm_k, 0, ky, kz, fb);
          tma_load_3d(dst + kHalfBytes, &tm_k, 64, ky, kz, fb);
          if (++st == kStages) { st = 0; st_phase ^= 1u; }
        }
        pos = advance(pos, r, REV);
        ++run_idx;
      }
     }
      if (!ok) {
        // give loads already in flight a bounded chance to land before the CTA's shared memory goes away
        const unsigned long long t0 = now_ns();
        for (int s2 = 0; s2 < kStages; ++s2) {
          const int last = it - 1 - ((it - 1 - s2) % kStages + kStages) % kStages;   // last issue into stage s2
          if (it == 0 || last < 0) continue;
          while (!mbar_try(full_bar(s2), (last / kStages) & 1) && now_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1 || warp == 2) {
    // ---------------- MMA issuers ----------------
    // Two threads take alternate tiles.  Issuing a tile's MMAs blocks the thread for about as long as the
    // tensor pipe needs them; with one issuer the waits and bookkeeping between two tiles would leave the pipe
    // idle, with two the other thread is already past its waits and its MMAs queue up right behind.
    if (lane == 0) {
      const int me = warp - 1;
      const uint32_t idesc1 = instr_desc(128, kTileKeys), idesc2 = instr_desc(kTileKeys, R);
      // descriptor of the k-step ks of a tile = descriptor of the tile + (byte offset >> 4); the address field
      // cannot carry out of its 14 bits because shared memory ends below 256 KB
      const uint64_t q_desc0 = smem_desc(q_smem), k_desc0 = smem_desc(k_smem);
      const uint64_t q_hi = (uint64_t)(q_half_bytes >> 4), k_hi = (uint64_t)(kHalfBytes >> 4);
      int it = 0, run_idx = 0, st = 0, b = 0;
      uint32_t st_phase = 0, b_phase = 0;
      uint64_t k_desc = k_desc0;
      uint32_t d0 = tmem_base;
      bool ok = true;
     for (int pass = kFirstPass; pass <= kLastPass && ok; ++pass) {
      const bool REV = pass == 2;
      const uint32_t idesc = pass == 1 ? idesc1 : idesc2;
      for (int pos = first_pos(REV); more(pos, REV) && ok;) {
        const Run r = locate(a, pos, begin, end, REV);
        ok = mbar_wait(qfull_bar, run_idx & 1, abort_flag);
        if (!ok) break;
        if (run_idx == 0 && me == 0) trace_mark(a.trace, 2);
        for (int i = 0; i < r.count; ++i, ++it) {
         if ((it & 1) == me) {
          ok = mbar_wait(full_bar(st), st_phase, abort_flag) && mbar_wait(acce_bar(b), b_phase ^ 1u, abort_flag);
          if (!ok) break;
          if (it == 0) trace_mark(a.trace, 3);
          tc_fence_after();
          if (pass == 1) {
            for (int mt = 0; mt < MT; ++mt) {
              const uint64_t qd = q_desc0 + (uint64_t)(mt * ((128 * 128) >> 4));
#pragma unroll
              for (int ks = 0; ks < 8; ++ks) {
                const uint64_t off = (uint64_t)((ks & 3) * 2);
                tc_mma(d0 + mt * 128, qd + (ks >> 2) * q_hi + off, k_desc + (ks >> 2) * k_hi + off, idesc, ks > 0);
              }
            }
          } else {
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint64_t off = (uint64_t)((ks & 3) * 2);
              tc_mma(d0, k_desc + (ks >> 2) * k_hi + off, q_desc0 + (ks >> 2) * q_hi + off, idesc, ks > 0);
            }
          }
          tc_commit(empty_bar(st));       // K stage free once these MMAs have read it
          tc_commit(accf_bar(b));         // accumulator ready for the epilogue
         }
          k_desc += (uint64_t)(kStageBytes >> 4);
          if (++st == kStages) { st = 0; st_phase ^= 1u; k_desc = k_desc0; }
          d0 += (uint32_t)buf_cols;
          if (++b == n_bufs) { b = 0; b_phase ^= 1u; d0 = tmem_base; }
        }
        tc_commit(qempty_bar);            // Q tile free once the run's MMAs (of both issuers) are done
        pos = advance(pos, r, REV);
        ++run_idx;
      }
     }
      if (!ok) {
        // gave up: the MMAs this thread has issued must be through before the accumulators are released
        tc_commit(drain_bar(me));
        const unsigned long long t0 = now_ns();
        while (!mbar_try(drain_bar(me), 0) && now_ns() - t0 < kWaitLimitNs) {}
      }
    }
  } else if (warp >= 4) {
    // ---------------- epilogue: two warpgroups, alternating tiles ----------------
    const int et = tid - 128;                   // 0..255
    const int wg = et >> 7;                     // warpgroup 0 / 1
    const int row = et & 127;                   // TMEM lane this thread reads
    const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
    const float sc = a.scale_log2;
    const float inv_g = 1.0f / (float)a.G;
    int it = 0, run_idx = 0;
    bool ok = true;
   for (int pass = kFirstPass; pass <= kLastPass; ++pass) {
    const bool REV = pass == 2;
    if (MODE == 3 && pass == 2) {
      // every CTA's row statistics must be in memory before any row's log-sum-exp is formed
      epi_bar();
      if (et == 0) trace_mark(a.trace, 5);
      if (et == 0 && ok) grid_barrier(&g_grid_arrivals[2 * a.barrier_slot], gridDim.x + (unsigned)a.barrier_extra, abort_flag);
      if (et == 0) trace_mark(a.trace, 6);
      epi_bar();
      ok = ok && *abort_flag == 0;
    }
    for (int pos = first_pos(REV); more(pos, REV);) {
      const Run r = locate(a, pos, begin, end, REV);
      const int seg = r.s * a.n_kv_heads + r.g;
      const int first_cta = r.seg_tile0 / a.tiles_per_cta;
      float m_run[2] = {0.f, 0.f}, z_run[2] = {0.f, 0.f};      // reference 0: see the fast path below
      float* lse = stats + 256 * (run_idx & 1);
      if (pass == 2) {
        // merge the per-CTA partials of this segment into the rows' log-sum-exp (log2 units)
        const int n_slots = (r.seg_tile0 + r.tiles_seg - 1) / a.tiles_per_cta - first_cta + 1;
        // With R <= 128 two neighbouring lanes share a row (even / odd slots) and combine through a shuffle.
        {
          const int halves = 2 * R <= kEpiThreads ? 2 : 1;
          const int rr = halves == 2 ? ((et >> 1) < R ? (et >> 1) : -1) : (et < R ? et : -1);
          const int half = halves == 2 ? (et & 1) : 0;
          float l2;
          if (a.lse.lse_opt) {                                            // the caller's row statistics
            l2 = rr >= 0 ? a.lse.caller_lse(r.s, r.g, rr, a.G, a.window, a.q_head_inner != 0) : 0.f;
          } else {
            const bool has_win = a.lse.win_m != nullptr && rr >= 0;
            l2 = merged_row_lse(a.part_m + (long long)seg * a.slot_stride * R, a.part_z + (long long)seg * a.slot_stride * R,
                                n_slots, R, rr, half, halves, has_win,
                                has_win ? a.lse.win_m[(long long)seg * R + rr] : 0.f,
                                has_win ? a.lse.win_z[(long long)seg * R + rr] : 0.f);
          }
          if (half == 0 && rr >= 0) lse[rr] = l2;
        }
        epi_bar();
        if (et == 0 && pass == 2 && pos == first_pos(true)) trace_mark(a.trace, 7);
      }
      for (int i = 0; i < r.count; ++i, ++it) {
        if ((it & 1) != wg) continue;
        const int b = it & (n_bufs - 1);                // n_bufs is 4 or 2
        if (ok) ok = mbar_wait(accf_bar(b), (it >> (n_bufs == 4 ? 2 : 1)) & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok) != 0;         // the TMEM loads below need the whole warp
        if (!ok) continue;
        tc_fence_after();
        if (row == 0 && it < 28) trace_mark(a.trace, 8 + 2 * it);
        const int key0 = tile_of(r, i, REV) * kTileKeys;
        const uint32_t tb = tmem_base + lane_sel + (uint32_t)(b * buf_cols);
        uint32_t ra[32], rb[32];
        if (pass == 1) {
          const int n_valid = min(r.n_hist - key0, kTileKeys);
          for (int mt = 0; mt < MT; ++mt) {
            const uint32_t tcol = tb + mt * 128;
            float m = m_run[mt], z = z_run[mt];
            bool exact = n_valid < kTileKeys;
            if (!exact) {
              // Fast path: a fixed reference m (0 until a fallback moves it) instead of a running maximum -- any
              // reference gives the same log-sum-exp as long as nothing overflows and not everything underflows;
              // a non-finite or zero sum shows that, and the tile is then redone exactly.
              float zt = z;
              tc_ld32_issue(tcol, ra);
#pragma unroll 1
              for (int c0 = 0; c0 < kTileKeys; c0 += 64) {      // rolled: half the code to keep in the instruction cache
                tc_ld_wait(ra);
                tc_ld32_issue(tcol + c0 + 32, rb);
                zt += sum_ex2_32(ra, sc, m);
                tc_ld_wait(rb);
                if (c0 + 64 < kTileKeys) tc_ld32_issue(tcol + c0 + 64, ra);
                zt += sum_ex2_32(rb, sc, m);
              }
              if (zt < INFINITY && zt > kTinySum) z = zt; else exact = true;
            }
            if (exact) tile_row_stats_exact(tcol, sc, n_valid, m, z);
            m_run[mt] = m; z_run[mt] = z;
          }
        } else {
          float acc = 0.f;
          tc_ld32_issue(tb, ra);
#pragma unroll 1
          for (int c0 = 0; c0 < R; c0 += 64) {
            tc_ld_wait(ra);
            if (c0 + 32 < R) tc_ld32_issue(tb + c0 + 32, rb);
            {
              float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
              for (int e = 0; e < 32; e += 4) {
                const float4 l4 = *reinterpret_cast<const float4*>(lse + c0 + e);
                s0 += ex2(fmaf(__uint_as_float(ra[e]), sc, -l4.x));
                s1 += ex2(fmaf(__uint_as_float(ra[e + 1]), sc, -l4.y));
                s2 += ex2(fmaf(__uint_as_float(ra[e + 2]), sc, -l4.z));
                s3 += ex2_fma(fmaf(__uint_as_float(ra[e + 3]), sc, -l4.w), false);
              }
              acc += (s0 + s1) + (s2 + s3);
            }
            if (c0 + 32 < R) {
              tc_ld_wait(rb);
              if (c0 + 64 < R) tc_ld32_issue(tb + c0 + 64, ra);
              float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
              for (int e = 0; e < 32; e += 4) {
                const float4 l4 = *reinterpret_cast<const float4*>(lse + c0 + 32 + e);
                s0 += ex2(fmaf(__uint_as_float(rb[e]), sc, -l4.x));
                s1 += ex2(fmaf(__uint_as_float(rb[e + 1]), sc, -l4.y));
                s2 += ex2(fmaf(__uint_as_float(rb[e + 2]), sc, -l4.z));
                s3 += ex2_fma(fmaf(__uint_as_float(rb[e + 3]), sc, -l4.w), false);
              }
              acc += (s0 + s1) + (s2 + s3);
            }
          }
          // The accumulator is in registers now: hand its TMEM buffer back before the vote leaves for global
          // memory (the arrive has release semantics and would otherwise wait for that store).
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(acce_bar(b));
          const int j = key0 + row;
          if (j < r.n_hist) a.vote[a.tab.hist_at(r.s) * a.n_kv_heads + (long long)r.g * r.n_hist + j] = acc * inv_g;
        }
        if (pass == 1) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(acce_bar(b));
        }
        if (row == 0 && it < 28) trace_mark(a.trace, 9 + 2 * it);
      }
      if (pass == 1) {
        // combine the two warpgroups' statistics and publish this CTA's partial for the segment
        const int slot = blockIdx.x - first_cta;
        for (int mt = 0; mt < MT; ++mt) {
          if (wg == 1) { stat_m[row] = m_run[mt]; stat_z[row] = z_run[mt]; }
          epi_bar();
          if (wg == 0) {
            const int rr = mt * 128 + row;
            if (rr < R) {
              const float m1 = stat_m[row], z1 = stat_z[row];
              const bool h0 = z_run[mt] > 0.f, h1 = z1 > 0.f;      // a warpgroup without a tile in this run has z = 0
              const float M = h0 && h1 ? fmaxf(m_run[mt], m1) : (h0 ? m_run[mt] : m1);
              float Z = 0.f;
              if (h0) Z += z_run[mt] * ex2(m_run[mt] - M);
              if (h1) Z += z1 * ex2(m1 - M);
              a.part_m[((long long)seg * a.slot_stride + slot) * R + rr] = M;
              a.part_z[((long long)seg * a.slot_stride + slot) * R + rr] = Z;
            }
          }
          epi_bar();
        }
      }
      pos = advance(pos, r, REV);
      ++run_idx;
    }
   }
  }

  tc_fence_before();
  __syncthreads();
  if (abort_sh && tid == 0 && a.status) atomicExch(a.status, (int)SLKV_ERR_DEVICE_TIMEOUT);
  if (tid == 0) trace_mark(a.trace, 4);
  if (MODE == 3 && tid == 0) {
    // every thread of this CTA is past the grid barrier (the CTA-wide barrier above): the last CTA out cleans the slot
    unsigned* slot = &g_grid_arrivals[2 * a.barrier_slot];
    unsigned prev;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(prev) : "l"(slot + 1) : "memory");
    if (prev == gridDim.x - 1) {
      slot[0] = 0;
      slot[1] = 0;
      __threadfence();
    }
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// lse_out[s][h][i] from the per-CTA statistics pass 1 left (tensor layout), in the units out_scale converts to.
__global__ void __launch_bounds__(kEpiThreads)
k_merge_lse_tensor(const __grid_constant__ TcArgs a, float* __restrict__ lse_out, float out_scale) {
  pdl_launch_dependents();
  pdl_wait();
  const int seg = blockIdx.x, s = seg / a.n_kv_heads, g = seg - s * a.n_kv_heads;
  const int n_hist = a.tab.cu_at(s + 1) - a.tab.cu_at(s) - a.window;
  if (n_hist <= 0) return;
  const int R = a.R, et = threadIdx.x;
  const int tiles_seg = a.tab.tile_at(s + 1) - a.tab.tile_at(s);
  const int seg_tile0 = a.n_kv_heads * a.tab.tile_at(s) + g * tiles_seg;
  const int first_cta = seg_tile0 / a.tiles_per_cta;
  const int n_slots = (seg_tile0 + tiles_seg - 1) / a.tiles_per_cta - first_cta + 1;
  const int halves = 2 * R <= kEpiThreads ? 2 : 1;
  const int rr = halves == 2 ? ((et >> 1) < R ? (et >> 1) : -1) : (et < R ? et : -1);
  const int half = halves == 2 ? (et & 1) : 0;
  const bool has_win = a.lse.win_m != nullptr && rr >= 0;
  const float l2 = merged_row_lse(a.part_m + (long long)seg * a.slot_stride * R, a.part_z + (long long)seg * a.slot_stride * R,
                                  n_slots, R, rr, half, halves, has_win,
                                  has_win ? a.lse.win_m[(long long)seg * R + rr] : 0.f,
                                  has_win ? a.lse.win_z[(long long)seg * R + rr] : 0.f);
  if (half == 0 && rr >= 0) {
    const int hh = a.q_head_inner ? rr % a.G : rr / a.window;
    const int i = a.q_head_inner ? rr / a.G : rr - hh * a.window;
    lse_out[((long long)s * a.lse.n_q_heads + g * a.G + hh) * a.window + i] = l2 * out_scale;
  }
}

// ---- host side ----------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

int sm_count() {
  static thread_local int dev_cached = -1, n = 0;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (dev != dev_cached) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n = 148;
    dev_cached = dev;
  }
  return n;
}

struct Schedule { int total_tiles, tiles_per_cta, n_cta; };

// One-shot diagnostic: the next launch of this thread whose CTAs wait for one another expects one arrival too many.
thread_local int g_expire_next_wait = 0;

// Timeline tracing (diagnostics): a caller-owned device buffer, two halves (pass 1, pass 2).
thread_local unsigned long long* g_trace = nullptr;
thread_local size_t g_trace_bytes = 0;
unsigned long long* trace_buffer(int pass, int n_cta) {
  const size_t need = (size_t)n_cta * kTraceSlots * sizeof(unsigned long long);
  if (!g_trace || g_trace_bytes < 2 * need) return nullptr;
  return g_trace + (pass - 1) * (size_t)n_cta * kTraceSlots;
}

Schedule schedule_of(const Problem& pb, const int32_t* cu_host) {
  long long tiles = 0;
  for (int s = 0; s < pb.p.n_seqs; ++s) {
    long long nh = (long long)cu_host[s + 1] - cu_host[s] - pb.p.window;
    if (nh > 0) tiles += (nh + kTileKeys - 1) / kTileKeys;
  }
  Schedule sc;
  sc.total_tiles = (int)(tiles * pb.p.n_kv_heads);
  int sms = sm_count();
  if (pb.max_score_ctas > 0 && pb.max_score_ctas < sms) sms = pb.max_score_ctas;
  sc.tiles_per_cta = sc.total_tiles > 0 ? (sc.total_tiles + sms - 1) / sms : 1;
  // A CTA whose range straddles two segments reloads Q in mid-stream (a pipeline bubble of a few microseconds) and
  // holds everybody else up wherever CTAs wait for one another.  When all segments have the same number of tiles
  // and a share per CTA at most 1/15 larger divides it, the ranges line up with the segments (more than that costs
  // more than the bubbles).
  if (pb.p.n_seqs > 0 && sc.total_tiles > 0) {
    const long long per_seg = tiles / pb.p.n_seqs;
    bool equal = per_seg * pb.p.n_seqs == tiles;
    for (int s = 0; s < pb.p.n_seqs && equal; ++s) {
      long long nh = (long long)cu_host[s + 1] - cu_host[s] - pb.p.window;
      equal = nh > 0 && (nh + kTileKeys - 1) / kTileKeys == per_seg;
    }
    if (equal && per_seg >= sc.tiles_per_cta)
      for (int t = sc.tiles_per_cta; (t - sc.tiles_per_cta) * 15 <= sc.tiles_per_cta; ++t)      // at most 1/15 more tiles
        if (per_seg % t == 0) { sc.tiles_per_cta = t; break; }
  }
  sc.n_cta = sc.total_tiles > 0 ? (sc.total_tiles + sc.tiles_per_cta - 1) / sc.tiles_per_cta : 0;
  return sc;
}

}  // namespace

void set_tensor_trace(void* dev_buf, size_t bytes) {
  g_trace = static_cast<unsigned long long*>(dev_buf);
  g_trace_bytes = bytes;
}

bool tensor_path_supported(const slkv_params& p) {
  if (p.dtype != SLKV_BF16 || p.head_dim != 128) return false;
  const int G = p.n_q_heads / p.n_kv_heads, R = G * p.window;
  if (R % 32 != 0 || R > 256 || p.window > 256 || G > 256) return false;
  return encode_fn() != nullptr;
}

// Row order inside the Q tile: the query heads of a group next to each other (r = i*G + hh) when the head stride is
// the smaller one, else the window rows (r = hh*window + i).
bool tensor_q_head_inner(const slkv_params& p) { return p.q_stride_head <= p.q_stride_row; }

int tensor_slot_stride(const Problem& pb) { return (pb.max_hist + kTileKeys - 1) / kTileKeys + 2; }

cudaError_t plan_score_tensor(const Problem& pb, const int32_t* cu_host, int32_t* status, TcPlan* plan) {
  plan->n_cta = 0;
  if (pb.max_hist <= 0) return cudaSuccess;
  EncodeTiledFn enc = encode_fn();
  if (!enc) return cudaErrorNotSupported;
  const slkv_params& p = pb.p;
  const Schedule sc = schedule_of(pb, cu_host);
  if (sc.n_cta == 0) return cudaSuccess;
  CUtensorMap& tm_q = plan->tm_q;
  CUtensorMap& tm_k = plan->tm_k;
  TcArgs& a = plan->a;

  // Tensor-map dimensions go from the smallest stride to the largest.  The order of the G*w query rows
  // inside the Q tile follows from it (head-fastest or window-row-fastest); the scores do not depend on it.
  const int q_head_inner = tensor_q_head_inner(p) ? 1 : 0;
  const int k_head_inner = p.k_stride_head <= p.k_stride_tok;
  {
    cuuint64_t dims[4] = {(cuuint64_t)p.head_dim, (cuuint64_t)p.window, (cuuint64_t)p.n_q_heads, (cuuint64_t)p.n_seqs};
    cuuint64_t strides[3] = {(cuuint64_t)p.q_stride_row * 2, (cuuint64_t)p.q_stride_head * 2, (cuuint64_t)p.q_stride_seq * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)p.window, (cuuint32_t)pb.G, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    if (q_head_inner) {
      cuuint64_t t = dims[1]; dims[1] = dims[2]; dims[2] = t;
      t = strides[0]; strides[0] = strides[1]; strides[1] = t;
      cuuint32_t b = box[1]; box[1] = box[2]; box[2] = b;
    }
    if (enc(&tm_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(pb.q), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
  }
  {
    cuuint64_t dims[3] = {(cuuint64_t)p.head_dim, (cuuint64_t)p.n_kv_heads, (cuuint64_t)pb.total_tokens};
    cuuint64_t strides[2] = {(cuuint64_t)p.k_stride_head * 2, (cuuint64_t)p.k_stride_tok * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)kTileKeys};
    cuuint32_t estr[3] = {1, 1, 1};
    if (!k_head_inner) {
      cuuint64_t t = dims[1]; dims[1] = dims[2]; dims[2] = t;
      t = strides[0]; strides[0] = strides[1]; strides[1] = t;
      cuuint32_t b = box[1]; box[1] = box[2]; box[2] = b;
    }
    if (enc(&tm_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(pb.k), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
  }

  a.tab = pb.tab;
  a.part_m = pb.part_m; a.part_z = pb.part_z; a.vote = pb.vote; a.status = status;
  a.lse = lse_source_of(pb);
  a.trace = nullptr;
  a.barrier_slot = 0;
  a.barrier_extra = 0;
  a.fresh_inputs = 0;
  a.n_seqs = p.n_seqs; a.n_kv_heads = p.n_kv_heads; a.G = pb.G; a.window = p.window; a.R = pb.R;
  a.MT = (pb.R + 127) / 128;
  a.q_head_inner = q_head_inner; a.k_head_inner = k_head_inner;
  a.slot_stride = pb.n_chunks;
  a.tiles_per_cta = sc.tiles_per_cta; a.total_tiles = sc.total_tiles;
  a.scale_log2 = kLog2e / sqrtf((float)p.head_dim);

  const size_t q_bytes = (size_t)a.MT * 2 * 128 * 128;
  a.n_stages = (int)((kSmemLimit - kTailBytes - q_bytes) / kStageBytes);
  if (a.n_stages > kMaxStages) a.n_stages = kMaxStages;
  plan->n_cta = sc.n_cta;
  return cudaSuccess;
}

unsigned long long* tensor_trace_buffer(int half, int n_cta) { return trace_buffer(half + 1, n_cta); }

void expire_next_wait(int on) { g_expire_next_wait = on; }
int take_expire_next_wait() { const int v = g_expire_next_wait; g_expire_next_wait = 0; return v; }

cudaError_t launch_merge_lse_tensor(const Problem& pb, const int32_t* cu_host, float* lse_out, cudaStream_t st,
                                    int* launches) {
  TcPlan plan;
  cudaError_t pe = plan_score_tensor(pb, cu_host, nullptr, &plan);
  if (pe != cudaSuccess || plan.n_cta == 0) return pe;
  LaunchScope scope(KID_MERGE_LSE, st, launches);
  return launch_pdl(k_merge_lse_tensor, dim3(pb.n_seg), dim3(kEpiThreads), 0, st, 1, plan.a, lse_out, lse_out_scale(pb));
}


cudaError_t launch_score_tensor(const Problem& pb, const int32_t* cu_host, int32_t* status, int passes,
                                cudaStream_t st, int* launches) {
  TcPlan plan;
  cudaError_t pe = plan_score_tensor(pb, cu_host, status, &plan);
  if (pe != cudaSuccess || plan.n_cta == 0) return pe;
  const CUtensorMap& tm_q = plan.tm_q;
  const CUtensorMap& tm_k = plan.tm_k;
  TcArgs& a = plan.a;
  struct { int n_cta; } sc = {plan.n_cta};
  const size_t q_bytes = (size_t)a.MT * 2 * 128 * 128;
  const size_t smem = q_bytes + (size_t)a.n_stages * kStageBytes + kTailBytes;
  static thread_local int configured_dev = -1;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (configured_dev != dev) {
    e = cudaFuncSetAttribute(k_score_tc<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_score_tc<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
    if (e != cudaSuccess) return e;
    configured_dev = dev;
  }
  // Both passes in one cooperative launch when the device takes it (all CTAs resident: the kernel has a
  // grid-wide barrier); otherwise two launches.
  static thread_local int fused_state[64] = {};       // per device: 0 untried, 1 cooperative + dependent launch,
                                                      // 2 cooperative only, -1 not available
  int& fs = fused_state[dev < 64 ? dev : 0];
  if (fs == 0) {
    int coop = 0;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) fs = -1;
    else if (cudaFuncSetAttribute(k_score_tc<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess)
      fs = -1;
    else fs = 1;
  }
  if (passes == 3 && fs > 0 && sc.n_cta <= sm_count()) {
    for (int attempt = 0; attempt < 2 && fs > 0; ++attempt) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(sc.n_cta);
      cfg.blockDim = dim3(kThreads);
      cfg.dynamicSmemBytes = smem;
      cfg.stream = st;
      cudaLaunchAttribute attr[2];
      int n = 0;
      attr[n].id = cudaLaunchAttributeCooperative;
      attr[n].val.cooperative = 1;
      ++n;
      if (fs == 1) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
      }
      cfg.attrs = attr;
      cfg.numAttrs = n;
      a.trace = trace_buffer(1, sc.n_cta);
      static std::atomic<unsigned> launch_seq{0};
      a.barrier_slot = (int)(launch_seq.fetch_add(1) % kBarrierSlots);
      a.barrier_extra = g_expire_next_wait ? 1 : 0;
      g_expire_next_wait = 0;
      cudaError_t le;
      {
        LaunchScope scope(KID_SCORE_FUSED, st, launches);
        le = cudaLaunchKernelEx(&cfg, k_score_tc<3>, tm_q, tm_k, a);
      }
      if (le == cudaSuccess) return cudaSuccess;
      (void)cudaGetLastError();                       // not a sticky error: the launch was refused
      --*launches;
      fs = fs == 1 ? 2 : -1;                          // try without dependent launch, then give up on fusing
    }
  }
  if (passes & 1) {
    LaunchScope scope(KID_SCORE_LSE, st, launches);
    a.trace = trace_buffer(1, sc.n_cta);
    e = launch_pdl(k_score_tc<1>, dim3(sc.n_cta), dim3(kThreads), smem, st, 1, tm_q, tm_k, a);
    if (e != cudaSuccess) return e;
  }
  if (!(passes & 2)) return cudaSuccess;
  LaunchScope scope(KID_SCORE_VOTE, st, launches);
  a.fresh_inputs = (passes & 1) ? 0 : 1;              // a vote pass on its own is the first to read Q and K
  a.trace = trace_buffer(2, sc.n_cta);
  return launch_pdl(k_score_tc<2>, dim3(sc.n_cta), dim3(kThreads), smem, st, 1, tm_q, tm_k, a);
}

}  // namespace slkv
