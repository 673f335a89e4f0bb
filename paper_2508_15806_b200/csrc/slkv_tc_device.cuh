// Device-side building blocks of the tensor-core score kernels (Sec. 3.4, Eq. 7; Algorithm 3): PTX wrappers for
// mbarriers, TMA loads, tcgen05 MMA / TMEM loads, the 2^x arithmetic, the tile schedule.  Included by the .cu
// files that hold the kernels; everything here has internal linkage.
#pragma once
#include <cuda.h>

#include "slkv_internal.cuh"

namespace slkv {

namespace {

constexpr int kTileKeys = 128;                 // keys per tile (MMA N in pass 1, M in pass 2)
constexpr int kMaxStages = 6;                  // K tiles in flight in shared memory (as many as fit beside Q)
constexpr int kHalfBytes = kTileKeys * 128;    // one 64-element (128-byte) half of a 128-row tile
constexpr int kStageBytes = 2 * kHalfBytes;    // 32 KB
constexpr int kTailBytes = 512 + 2048;         // mbarriers + flags, then 512 floats of row statistics
constexpr int kSmemLimit = 227 * 1024;         // dynamic shared memory a CTA can have
constexpr int kThreads = 384;                  // warps 0-3: TMA, MMA, 2 idle; warps 4-11: epilogue
constexpr int kEpiThreads = 256;
constexpr int kTraceSlots = 64;               // per CTA: 0 start, 1 set-up done, 2 Q landed, 3 first K landed,
                                               // 4 end; 5 / 6 grid barrier reached / passed, 7 first log-sum-exp merged; 8+2i / 9+2i = epilogue of the
                                               // CTA's i-th tile begins / ends.  Two-layer kernel: 0 start, 1 / 7 stream A / B
                                               // past its wait for the launch before, 2 first accumulator of A ready,
                                               // 3 first log-sum-exps of B merged, 5 / 6 epilogue of A / B done, 4 end,
                                               // 8+2j / 9+2j layer j published by A / begun by B, 60 / 61 SM cycle counter at start / end
// A row sum under the fixed reference that is not above this has underflowed (terms below fp32's range are flushed
// to zero, or clamped to 2^-125 on the polynomial path): the exact path then moves the reference.
constexpr float kTinySum = 1e-30f;
constexpr unsigned long long kWaitLimitNs = 1000ull * 1000ull * 1000ull;   // 1 s per wait


// ---- PTX wrappers -------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity), "r"(100u) : "memory");    // may sleep up to 0.1 us: a waiting thread must
                                                                   // not eat the issue slots of the epilogue warps
  return ok != 0;
}
__device__ __forceinline__ unsigned long long now_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void trace_mark(const unsigned long long* base, int slot) {
  if (base) const_cast<unsigned long long*>(base)[(size_t)blockIdx.x * kTraceSlots + slot] = now_ns();
}
// Waits for the phase with the given parity.  false = gave up (limit reached or another thread did).
// backoff_ns > 0: sleep that long between polls, so that a waiting warp leaves the issue slots to the working ones.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned backoff_ns = 0) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = now_ns();
  for (unsigned it = 1;; ++it) {
    if (backoff_ns) __nanosleep(backoff_ns);
    if (mbar_try(bar, parity)) return true;
    if ((it & 63u) == 0) {
      if (*abort_flag) return false;
      if (now_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
    }
  }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
// The same load with an L2 eviction policy (from createpolicy) for the lines it touches.
__device__ __forceinline__ void tma_load_3d_hint(uint32_t dst, const CUtensorMap* tm, int x, int y, int z, uint32_t bar,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3, %4}], [%5], %6;"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(z), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, int x, int y, int z, int w,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(z), "r"(w), "r"(bar) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// 2^x on the FMA and integer pipes instead of the special-function unit, which is the busiest pipe of both
// passes (one exponential per query row and key): x = n + f with n = round(x), 2^f by a degree-4 minimax
// polynomial on [-0.5, 0.5] (relative error 2.7e-6 in fp32 Horner form), n added into the exponent field.
// x is clamped to [-125, 128.5]: below, the result is 2^-125 at most (negligible in any sum that holds a term
// near 1); above, the exponent field overflows to Inf/NaN, which the caller's overflow check catches.
// One exponential in four goes this way; the split balances the pipes' issue slots.
__device__ __forceinline__ float ex2_fma(float x, bool clamp_hi) {
  x = fmaxf(x, -125.f);
  if (clamp_hi) x = fminf(x, 128.5f);
  const float t = x + 12582912.f;                    // 1.5 * 2^23: round(x) lands in the low mantissa bits
  const float f = x - (t - 12582912.f);
  float p = fmaf(0.009570101276040077f, f, 0.05591785907745361f);
  p = fmaf(p, f, 0.240247443318367f);
  p = fmaf(p, f, 0.6931217908859253f);
  p = fmaf(p, f, 0.9999992847442627f);
  return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}
// Issues a TMEM load of 32 consecutive columns of this thread's lane; the registers are valid only after
// tc_ld_wait on the same array.
__device__ __forceinline__ void tc_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
// The same for 16 columns (half the registers of a round; used where more warps share the register file).
__device__ __forceinline__ void tc_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_ld_wait16(uint32_t (&r)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
      : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
        "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]) :: "memory");
}
// Waits for this thread's outstanding TMEM loads; naming the registers keeps their uses behind the wait.
__device__ __forceinline__ void tc_ld_wait(uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.wait::ld.sync.aligned;"
      : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
        "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]),
        "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
        "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
      :: "memory");
}
__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }

// K-major, 128-byte-swizzled operand: rows 128 bytes apart, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// D fp32, A and B bf16, both K-major, M x N tile
__device__ __forceinline__ uint32_t instr_desc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Merges the per-CTA partial statistics [slot][row] of one row of a segment (pm / pz point at the segment's first
// slot) into the row's log-sum-exp in log2 units, the window keys' statistics (wm, wz) folded in when has_win.  With
// halves == 2 two neighbouring lanes share a row (even / odd slots) and combine through a shuffle, so all 32 lanes
// of a warp must call it; lanes without a row pass rr < 0.  Every thread has all its loads in flight before it uses
// one.  One definition for every kernel that merges, so that they agree bit for bit.
__device__ __forceinline__ float merged_row_lse(const float* pm, const float* pz, int n_slots, int R, int rr, int half,
                                                int halves, bool has_win, float wm, float wz) {
  float M = -INFINITY, Z = 0.f;
  if (rr >= 0) {
    pm += rr;                                                              // [segment][slot][row]
    pz += rr;
    for (int c0 = half; c0 < n_slots; c0 += 12 * halves) {
      float m12[12], z12[12];
#pragma unroll
      for (int u = 0; u < 12; ++u) {
        const int c = c0 + u * halves;
        const bool in = c < n_slots;
        m12[u] = in ? __ldcg(pm + (long long)c * R) : -INFINITY;
        z12[u] = in ? __ldcg(pz + (long long)c * R) : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 12; ++u)
        if (z12[u] > 0.f) {                                                // empty partials carry z = 0
          const float Mn = fmaxf(M, m12[u]);
          Z = fmaf(Z, ex2(M - Mn), __fmul_rn(z12[u], ex2(m12[u] - Mn)));   // ex2(-inf) = 0 covers the first term;
                                                                           // explicit rounding: the same in every kernel
          M = Mn;
        }
    }
  }
  if (halves == 2) {                                                       // uniform over the warp
    const float M1 = __shfl_xor_sync(0xffffffffu, M, 1), Z1 = __shfl_xor_sync(0xffffffffu, Z, 1);
    const float Mn = fmaxf(M, M1);
    float Zt = 0.f;
    if (M > -INFINITY) Zt = __fmul_rn(Z, ex2(M - Mn));
    if (M1 > -INFINITY) Zt = __fadd_rn(Zt, __fmul_rn(Z1, ex2(M1 - Mn)));
    M = Mn; Z = Zt;
  }
  if (has_win && wz > 0.f) {
    const float Mn = fmaxf(M, wm);
    Z = __fadd_rn(M > -INFINITY ? __fmul_rn(Z, ex2(M - Mn)) : 0.f, __fmul_rn(wz, ex2(wm - Mn)));
    M = Mn;
  }
  return __fadd_rn(M, log2f(Z));
}

struct Run { int s, g, t0, count, n_hist, seg_tile0, tiles_seg; };

// A run = consecutive tiles of one segment inside the CTA's range [begin, end).  Forward walks (pass 1)
// name a run by its first tile, backward walks (pass 2) by its last one.
__device__ __forceinline__ Run locate(const TcArgs& a, int pos, int begin, int end, bool REV) {
  int lo = 0, hi = a.n_seqs;                       // last s with Hkv*tile_off[s] <= pos
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (a.n_kv_heads * a.tab.tile_at(mid) <= pos) lo = mid; else hi = mid;
  }
  Run r;
  r.s = lo;
  r.tiles_seg = a.tab.tile_at(lo + 1) - a.tab.tile_at(lo);
  const int rel = pos - a.n_kv_heads * a.tab.tile_at(lo);
  r.g = rel / r.tiles_seg;
  const int t = rel - r.g * r.tiles_seg;
  r.seg_tile0 = pos - t;
  if (REV) {
    r.t0 = max(r.seg_tile0, begin) - r.seg_tile0;
    r.count = t - r.t0 + 1;
  } else {
    r.t0 = t;
    r.count = min(end - pos, r.tiles_seg - t);
  }
  r.n_hist = max(a.tab.cu_at(lo + 1) - a.tab.cu_at(lo) - a.window, 0);
  return r;
}

// sum_e 2^(v_e * sc - m) over 32 accumulator values, four independent chains
__device__ __forceinline__ float sum_ex2_32(const uint32_t (&r)[32], float sc, float m) {
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
  for (int e = 0; e < 32; e += 4) {
    s0 += ex2(fmaf(__uint_as_float(r[e]), sc, -m));
    s1 += ex2(fmaf(__uint_as_float(r[e + 1]), sc, -m));
    s2 += ex2(fmaf(__uint_as_float(r[e + 2]), sc, -m));
    s3 += ex2_fma(fmaf(__uint_as_float(r[e + 3]), sc, -m), true);
  }
  return (s0 + s1) + (s2 + s3);
}
// Adds one chunk of 32 accumulator values (the first nv of them) to a row's (reference m, sum z) pair exactly:
// the reference moves to the running maximum and the sum is rescaled.  Taken when the fixed-reference sum of the
// chunk over- or underflowed; works on the registers, so the accumulator may already be back with the tensor pipe.
__device__ __noinline__ void chunk_stats_exact(const uint32_t (&r)[32], float sc, int nv, float& m_io, float& z_io) {
  float mx = -INFINITY;
#pragma unroll
  for (int e = 0; e < 32; ++e)
    if (e < nv) mx = fmaxf(mx, __uint_as_float(r[e]) * sc);
  if (!(mx > -INFINITY)) return;                       // nothing valid (or only -inf scores)
  const float m_new = z_io > 0.f ? fmaxf(m_io, mx) : mx;
  float z = z_io > 0.f ? z_io * ex2(m_io - m_new) : 0.f;
#pragma unroll
  for (int e = 0; e < 32; ++e)
    if (e < nv) z += ex2(fmaf(__uint_as_float(r[e]), sc, -m_new));
  m_io = m_new; z_io = z;
}
__device__ __forceinline__ float max_32(const uint32_t (&r)[32], int n_valid_here) {
  float t[32];
#pragma unroll
  for (int e = 0; e < 32; ++e) t[e] = e < n_valid_here ? __uint_as_float(r[e]) : -INFINITY;
#pragma unroll
  for (int w = 16; w >= 1; w >>= 1)
#pragma unroll
    for (int e = 0; e < w; ++e) t[e] = fmaxf(t[e], t[e + w]);
  return t[0];
}

// Pass 1, exact path for one 128-row accumulator: running maximum and rescaled sum over the tile's first n_valid
// keys.  Used for a segment's ragged last tile and when the fast path over- or underflows.  A function of its
// own (not inlined) so that a CTA which will need it can run it once before the K stream starts: fetching
// these instructions for the first time while the stream saturates the memory system stalled the tile for
// microseconds.
__device__ __noinline__ void tile_row_stats_exact(uint32_t tcol, float sc, int n_valid, float& m_io, float& z_io) {
  uint32_t ra[32];
  float m = m_io, z = z_io;
#pragma unroll 1
  for (int c0 = 0; c0 < kTileKeys; c0 += 32) {
    if (c0 >= n_valid) break;
    tc_ld32_issue(tcol + c0, ra);
    tc_ld_wait(ra);
    // the reference a row starts with (0) is a guess, not a score: while nothing has been summed it gives way to
    // the first maximum seen, however low
    const float mx = max_32(ra, n_valid - c0) * sc;
    const float mn = z > 0.f ? fmaxf(m, mx) : mx;
    z = z > 0.f ? z * ex2(m - mn) : 0.f;
    m = mn;
    float zc = 0.f;
#pragma unroll
    for (int e = 0; e < 32; ++e)
      if (e < n_valid - c0) zc += ex2(fmaf(__uint_as_float(ra[e]), sc, -m));
    z += zc;
  }
  m_io = m; z_io = z;
}

}  // namespace
}  // namespace slkv
