// extern "C" entry points of libslkv: argument validation, workspace carve-up, launch sequencing.
// No step of the method runs here; every step is a kernel in the other translation units.
#include <cstring>
#include <mutex>
#include <vector>

#include "slkv_internal.cuh"

namespace slkv {
namespace {

thread_local int g_last_cuda_error = 0;
thread_local int g_last_launches = 0;

// ---- per-kernel timing (off by default) -----------------------------------------------------------
struct TimedLaunch { int kid; cudaEvent_t a, b; };
thread_local int g_prof_on = 0;          // 0 off, 1 every kernel (one stream), 2 the score kernels only (side streams kept)
thread_local std::vector<TimedLaunch>* g_prof = nullptr;      // records of the current thread
thread_local std::vector<cudaEvent_t>* g_prof_free = nullptr;

cudaEvent_t prof_event() {
  if (g_prof_free && !g_prof_free->empty()) {
    cudaEvent_t e = g_prof_free->back();
    g_prof_free->pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
  return e;
}

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

constexpr int kMinChunkKeys = 128;     // no score path uses smaller chunks (sizes the partial buffers)
constexpr int kMaxWindow = 256;
constexpr size_t kSimtSmemLimit = 192 * 1024;

int cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return SLKV_ERR_CUDA;
}

constexpr int kLaySlots = 2 * kPipeMaxLayers + 2;   // overlapped calls: layers in flight at once
struct Layout {
  size_t hist_off, tile_off, vote[kLaySlots], pooled, part_m[kLaySlots], part_z[kLaySlots], flags, gather_src[kLaySlots],
      win_m[kLaySlots], win_z[kLaySlots], total;
};

// Validates p and cu_seqlens_host and fills the host-known fields of `pb`.
int describe(const slkv_params* p, const int32_t* cu_host, Problem* pb) {
  if (!p || !cu_host) return SLKV_ERR_NULL_PTR;
  if (p->dtype != SLKV_F32 && p->dtype != SLKV_BF16) return SLKV_ERR_BAD_DTYPE;
  if (p->pool_mode != SLKV_POOL_MAX && p->pool_mode != SLKV_POOL_AVG) return SLKV_ERR_BAD_DTYPE;
  if (p->softmax_domain != SLKV_HISTORY && p->softmax_domain != SLKV_ALL_CAUSAL) return SLKV_ERR_BAD_DTYPE;
  if (p->lse_units != SLKV_LSE_LN && p->lse_units != SLKV_LSE_LOG2) return SLKV_ERR_BAD_DTYPE;
  if (p->history_only != 0 && p->history_only != 1) return SLKV_ERR_BAD_DTYPE;
  if (p->history_only && p->n_seqs != 1) return SLKV_ERR_BAD_SHAPE;
  if (p->score_path < SLKV_PATH_AUTO || p->score_path > SLKV_PATH_TENSOR) return SLKV_ERR_BAD_DTYPE;
  if (p->n_seqs < 1 || p->n_seqs > (1 << 20)) return SLKV_ERR_BAD_SHAPE;
  if (p->n_kv_heads < 1 || p->n_kv_heads > 65535 || p->n_q_heads < p->n_kv_heads ||
      p->n_q_heads % p->n_kv_heads != 0)
    return SLKV_ERR_BAD_SHAPE;
  if (p->head_dim != 64 && p->head_dim != 128) return SLKV_ERR_BAD_SHAPE;
  if (p->window < 1 || p->window > kMaxWindow) return SLKV_ERR_BAD_SHAPE;
  if (p->pool_kernel < 1 || p->pool_kernel % 2 == 0 || p->pool_kernel > 1025) return SLKV_ERR_BAD_SHAPE;
  const int elem = p->dtype == SLKV_F32 ? 4 : 2;
  const int64_t row = p->head_dim;
  if (p->k_stride_head < row || p->v_stride_head < row || p->q_stride_head < row ||
      p->k_stride_tok < row || p->v_stride_tok < row || p->q_stride_row < row || p->q_stride_seq < row)
    return SLKV_ERR_BAD_SHAPE;
  const int64_t strides[] = {p->k_stride_tok, p->k_stride_head, p->v_stride_tok, p->v_stride_head,
                             p->q_stride_seq, p->q_stride_row, p->q_stride_head};
  for (int64_t s : strides)
    if ((s * elem) % 16 != 0) return SLKV_ERR_BAD_ALIGN;
  if (cu_host[0] != 0) return SLKV_ERR_BAD_SHAPE;
  // History rows only: the kernels are told about a sequence of rows + window tokens whose last `window` rows they
  // never read (the window rows are only ever read as keys by the all-causal window statistics, which such a call
  // does not run); the K tensor map still ends at the rows that exist.
  const int64_t rows_given = cu_host[p->n_seqs];
  if (p->history_only && (cu_host[1] < 0 || (int64_t)cu_host[1] + p->window >= (1ll << 31))) return SLKV_ERR_BAD_SHAPE;
  const int32_t cu_virtual[2] = {0, p->history_only ? cu_host[1] + p->window : 0};
  if (p->history_only) cu_host = cu_virtual;
  int64_t total_hist = 0;
  int max_hist = 0;
  for (int s = 0; s < p->n_seqs; ++s) {
    int64_t len = (int64_t)cu_host[s + 1] - cu_host[s];
    if (len < 0) return SLKV_ERR_BAD_SHAPE;
    int64_t nh = len > p->window ? len - p->window : 0;
    total_hist += nh;
    if (nh > max_hist) max_hist = (int)nh;
  }
  const int64_t T = cu_host[p->n_seqs];
  if ((int64_t)p->n_kv_heads * T >= (1ll << 31)) return SLKV_ERR_BAD_SHAPE;
  std::memset(pb, 0, sizeof(*pb));
  pb->p = *p;
  pb->G = p->n_q_heads / p->n_kv_heads;
  pb->R = pb->G * p->window;
  pb->elem = elem;
  pb->max_hist = max_hist;
  pb->total_tokens = rows_given;
  if (p->history_only) {
    pb->p.softmax_domain = SLKV_HISTORY;
    pb->cu_virtual[0] = cu_virtual[0]; pb->cu_virtual[1] = cu_virtual[1];
  }
  pb->total_hist = total_hist;
  pb->n_seg = p->n_seqs * p->n_kv_heads;
  if (p->n_seqs <= kInlineSeqs) {
    pb->tab.n_inline = p->n_seqs;
    long long hacc = 0;
    int tacc = 0;
    for (int s = 0; s <= p->n_seqs; ++s) {
      pb->tab.cu[s] = cu_host[s];
      pb->tab.hist_off[s] = hacc;
      pb->tab.tile_off[s] = tacc;
      if (s < p->n_seqs) {
        long long nh = (long long)cu_host[s + 1] - cu_host[s] - p->window;
        if (nh < 0) nh = 0;
        hacc += nh;
        tacc += (int)((nh + 127) / 128);
      }
    }
  }
  if (pb->n_seg > 65535 * 16) return SLKV_ERR_BAD_SHAPE;
  if (pb->R > 1024) return SLKV_ERR_BAD_SHAPE;
  return SLKV_OK;
}

// Layers an overlapped call sequence keeps in flight: many where the score kernel takes lists of layers, three
// otherwise (one being scored, one being selected, one being gathered).
int overlapped_slots(const Problem& pb) {
  return tensor_path_supported(pb.p) && score_pipe_supported(pb) && pb.p.score_path != SLKV_PATH_SIMT ? kLaySlots : 3;
}

Layout layout_of(const Problem& pb, bool overlapped = false) {
  Layout L;
  size_t o = 0;
  L.hist_off = o; o = align_up(o + (size_t)(pb.p.n_seqs + 1) * sizeof(int64_t));
  L.tile_off = o; o = align_up(o + (size_t)(pb.p.n_seqs + 1) * sizeof(int32_t));
  // Overlapped calls keep many layers in flight (the score kernel takes a list of layers per launch, selections and
  // gathers trail behind): each has its own votes, source-row list and per-CTA row statistics.  Ordinary calls use
  // the first of each.
  const size_t votes = (size_t)pb.p.n_kv_heads * (size_t)pb.total_hist * sizeof(float);
  const int n_slots = overlapped ? overlapped_slots(pb) : 1;
  for (int i = 0; i < kLaySlots; ++i) {
    L.vote[i] = i < n_slots ? o : L.vote[0];
    if (i < n_slots) o = align_up(o + votes);
  }
  L.pooled = o; o = align_up(o + votes);
  const size_t nchunks = (size_t)(pb.max_hist + kMinChunkKeys - 1) / kMinChunkKeys + 2;
  const size_t parts = (size_t)pb.n_seg * pb.R * nchunks * sizeof(float);
  for (int i = 0; i < kLaySlots; ++i) {
    L.part_m[i] = i < n_slots ? o : L.part_m[0];
    if (i < n_slots) o = align_up(o + parts);
    L.part_z[i] = i < n_slots ? o : L.part_z[0];
    if (i < n_slots) o = align_up(o + parts);
  }
  L.flags = o; o = align_up(o + 8 * sizeof(int32_t));
  const size_t srcs = (size_t)pb.p.n_kv_heads * (size_t)pb.total_tokens * sizeof(int32_t);
  for (int i = 0; i < kLaySlots; ++i) {
    L.gather_src[i] = i < n_slots ? o : L.gather_src[0];
    if (i < n_slots) o = align_up(o + srcs);
  }
  // row statistics over the window keys (all-causal softmax domain): [n_seg][R] maxima and sums
  const size_t wins = (size_t)pb.n_seg * pb.R * sizeof(float);
  for (int i = 0; i < kLaySlots; ++i) {
    L.win_m[i] = i < n_slots ? o : L.win_m[0];
    if (i < n_slots) o = align_up(o + wins);
    L.win_z[i] = i < n_slots ? o : L.win_z[0];
    if (i < n_slots) o = align_up(o + wins);
  }
  L.total = o;
  return L;
}

// Picks the score path; SLKV_ERR_* when the requested one cannot take the shape.
int resolve_path(const Problem& pb, int* path) {
  int want = pb.p.score_path;
  const bool tensor_ok = tensor_path_supported(pb.p);
  if (want == SLKV_PATH_AUTO) want = tensor_ok ? SLKV_PATH_TENSOR : SLKV_PATH_SIMT;
  if (want == SLKV_PATH_TENSOR && !tensor_ok) return SLKV_ERR_BAD_DTYPE;
  if (want == SLKV_PATH_SIMT && simt_smem_bytes(pb) > kSimtSmemLimit) return SLKV_ERR_BAD_SHAPE;
  *path = want;
  return SLKV_OK;
}

// slot: which of the vote arrays / source-row lists / sets of row statistics (overlapped calls)
int bind_workspace(Problem* pb, void* ws, size_t ws_bytes, int path, bool overlapped = false, int slot = 0) {
  if (!ws) return SLKV_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) % kAlign != 0) return SLKV_ERR_BAD_ALIGN;
  Layout L = layout_of(*pb, overlapped);
  if (ws_bytes < L.total) return SLKV_ERR_WORKSPACE;
  unsigned char* b = static_cast<unsigned char*>(ws);
  pb->hist_off = reinterpret_cast<int64_t*>(b + L.hist_off);
  pb->tile_off = reinterpret_cast<int32_t*>(b + L.tile_off);
  pb->tab.tile_ptr = pb->tile_off;
  pb->tab.hist_ptr = reinterpret_cast<const long long*>(pb->hist_off);
  pb->vote = reinterpret_cast<float*>(b + L.vote[slot]);
  pb->pooled_ws = reinterpret_cast<float*>(b + L.pooled);
  pb->part_m = reinterpret_cast<float*>(b + L.part_m[slot]);
  pb->part_z = reinterpret_cast<float*>(b + L.part_z[slot]);
  pb->dev_flags = reinterpret_cast<int32_t*>(b + L.flags);
  pb->gather_src = reinterpret_cast<int32_t*>(b + L.gather_src[slot]);
  pb->win_m = reinterpret_cast<float*>(b + L.win_m[slot]);
  pb->win_z = reinterpret_cast<float*>(b + L.win_z[slot]);
  pb->chunk_keys = path == SLKV_PATH_TENSOR ? 128 : simt_chunk_keys();
  pb->n_chunks = path == SLKV_PATH_TENSOR ? tensor_slot_stride(*pb)
                                          : (pb->max_hist + pb->chunk_keys - 1) / pb->chunk_keys;
  if (pb->n_chunks < 1) pb->n_chunks = 1;
  return SLKV_OK;
}

bool aligned16(const void* p) { return reinterpret_cast<uintptr_t>(p) % 16 == 0; }

// The window keys' row statistics, where the softmax runs over all causally visible keys and the caller has not
// supplied the rows' log-sum-exp (Eq. 3-4 over the prefill attention's own key set).
int enqueue_window_stats(const Problem& pb, int path, cudaStream_t st, int* launches) {
  if (pb.lse_opt || pb.p.softmax_domain != SLKV_ALL_CAUSAL) return SLKV_OK;
  cudaError_t e = launch_window_stats(pb, path == SLKV_PATH_TENSOR && tensor_q_head_inner(pb.p), st, launches);
  if (e != cudaSuccess) return cuda_fail(e);
  return SLKV_OK;
}

// window votes of every history key (device pointers resolved); with the caller's row statistics the vote pass alone
int enqueue_votes(const Problem& pb, int path, const int32_t* cu_host, int32_t* status, cudaStream_t st,
                  int* launches) {
  int rc = enqueue_window_stats(pb, path, st, launches);
  if (rc != SLKV_OK) return rc;
  const int passes = pb.lse_opt ? 2 : 3;
  cudaError_t e = path == SLKV_PATH_TENSOR ? launch_score_tensor(pb, cu_host, status, passes, st, launches)
                                           : launch_score_simt(pb, passes, st, launches);
  if (e != cudaSuccess) return cuda_fail(e);
  return SLKV_OK;
}

// ---- overlapped calls ---------------------------------------------------------------------------------------
// The selection and the gather of a layer run on side streams while the score kernels of the following layers
// run on the caller's stream.  Where the two-layer score kernel takes the shape, a call enqueues pass 1 of its
// own layer together with pass 2 of the layer before (which stays "pending" until the next call or a join).
constexpr int kSlots = 2 * kPipeMaxLayers + 2;     // layers whose votes / source rows / row statistics are live at once
constexpr int kSideStreams = 9;   // after the last launch of a list the selections of its layers run side by side
struct PendingCall {
  bool valid = false;
  Problem pb;
  TcPlan plan;
  int slot = 0;
  const int32_t* budgets = nullptr;
  void* k_out = nullptr;
  void* v_out = nullptr;
  int64_t capacity = 0;
  int32_t* offsets = nullptr;
  int32_t* kept_idx = nullptr;
  float* pooled_opt = nullptr;
  int32_t* status = nullptr;
  cudaStream_t st = nullptr;
  std::vector<int32_t> cu_host;          // the call's cu_seqlens_host (the caller's copy is only valid during the call)
};
struct ShapeSig {                                  // calls in flight together must carve the workspace alike
  const void* ws = nullptr;
  size_t ws_bytes = 0;
  int n_seqs = 0, n_kv_heads = 0, R = 0, max_hist = 0, path = 0;
  int64_t total_hist = 0, total_tokens = 0;
  bool operator==(const ShapeSig& o) const {
    return ws == o.ws && ws_bytes == o.ws_bytes && n_seqs == o.n_seqs && n_kv_heads == o.n_kv_heads && R == o.R &&
           max_hist == o.max_hist && path == o.path && total_hist == o.total_hist && total_tokens == o.total_tokens;
  }
};
struct OverlapState {
  cudaStream_t side_select[kSideStreams] = {}, side_gather[kSideStreams] = {};   // slot s uses streams s % kSideStreams
  cudaEvent_t scored[kSlots] = {};       // recorded on the caller's stream after the vote pass of the slot's layer
  cudaEvent_t selected[kSlots] = {};     // recorded on a selection stream after the selection
  cudaEvent_t done[kSlots] = {};         // recorded on the gather stream after the gather
  bool in_flight[kSlots] = {};
  bool wait_done[kSlots] = {};           // the slot's next selection must first wait for the gather that had the slot
  unsigned seq = 0;
  std::vector<PendingCall> queue;        // layers whose score kernel is not launched yet (at most kPipeMaxLayers + 1)
  PendingCall pending;                   // pass 1 launched, pass 2 not
  std::vector<PendingCall> deferred;     // votes launched and `scored` recorded, selection and gather not enqueued yet
  ShapeSig sig;
};
// One state per (device, caller's stream): calls made on different streams (by different host threads, or by one)
// never share a queue, a slot or an event, so each stream's calls keep their own order whatever the others do.
constexpr int kMaxDevices = 64;
constexpr int kStatesPerDevice = 8;
struct DeviceStates {
  OverlapState st[kStatesPerDevice];
  cudaStream_t owner[kStatesPerDevice] = {};
  bool used[kStatesPerDevice] = {};
  unsigned long long last_use[kStatesPerDevice] = {};
  unsigned long long tick = 0;
};
DeviceStates g_overlap[kMaxDevices];
std::mutex g_overlap_mu;
constexpr int kSelectSmReserve = 16;              // SMs left to the selection kernels of the layers before

cudaError_t flush_pending(OverlapState* os, int* launches);

bool state_idle(const OverlapState& s) {
  if (!s.queue.empty() || s.pending.valid || !s.deferred.empty()) return false;
  for (int h = 0; h < kSlots; ++h)
    if (s.in_flight[h]) return false;
  return true;
}

// The state of overlapped calls made on `st` on the current device (g_overlap_mu held).  All eight in use by other
// streams: the one used longest ago is drained -- its queued layers go out and its own stream waits for what it has
// in flight, as a join on that stream would -- and handed over.
cudaError_t overlap_state(cudaStream_t st, OverlapState** out, int* launches) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  DeviceStates& d = g_overlap[dev];
  int idx = -1;
  for (int i = 0; i < kStatesPerDevice; ++i)
    if (d.used[i] && d.owner[i] == st) idx = i;
  if (idx < 0) {
    for (int i = 0; i < kStatesPerDevice && idx < 0; ++i)
      if (!d.used[i]) idx = i;
    if (idx < 0) {
      int oldest = 0, oldest_idle = -1;
      for (int i = 0; i < kStatesPerDevice; ++i) {
        if (d.last_use[i] < d.last_use[oldest]) oldest = i;
        if (state_idle(d.st[i]) && (oldest_idle < 0 || d.last_use[i] < d.last_use[oldest_idle])) oldest_idle = i;
      }
      idx = oldest_idle >= 0 ? oldest_idle : oldest;
      OverlapState& v = d.st[idx];
      e = flush_pending(&v, launches);
      for (int h = 0; h < kSlots && e == cudaSuccess; ++h)
        if (v.in_flight[h]) {
          e = cudaStreamWaitEvent(d.owner[idx], v.done[h], 0);
          v.in_flight[h] = false;
        }
      if (e != cudaSuccess) return e;
      v.sig = ShapeSig();
    }
    d.used[idx] = true;
    d.owner[idx] = st;
  }
  d.last_use[idx] = ++d.tick;
  OverlapState& s = d.st[idx];
  if (!s.side_gather[kSideStreams - 1]) {
    for (int i = 0; i < kSideStreams; ++i) {
      e = cudaStreamCreateWithFlags(&s.side_select[i], cudaStreamNonBlocking);
      if (e != cudaSuccess) return e;
      e = cudaStreamCreateWithFlags(&s.side_gather[i], cudaStreamNonBlocking);
      if (e != cudaSuccess) return e;
    }
    for (int h = 0; h < kSlots; ++h) {
      e = cudaEventCreateWithFlags(&s.scored[h], cudaEventDisableTiming);
      if (e != cudaSuccess) return e;
      e = cudaEventCreateWithFlags(&s.selected[h], cudaEventDisableTiming);
      if (e != cudaSuccess) return e;
      e = cudaEventCreateWithFlags(&s.done[h], cudaEventDisableTiming);
      if (e != cudaSuccess) return e;
    }
  }
  *out = &s;
  return cudaSuccess;
}

// Before a layer takes a slot: its vote array may still be read by the selection of the layer that had the slot,
// its source-row list by that layer's gather.
cudaError_t flush_deferred(OverlapState* os, int* launches);
cudaError_t claim_slot(OverlapState* os, int slot, cudaStream_t st, int* launches) {
  for (size_t i = 0; i < os->deferred.size(); ++i)
    if (os->deferred[i].slot == slot) {                              // its selection is not even enqueued yet
      cudaError_t e = flush_deferred(os, launches);
      if (e != cudaSuccess) return e;
      break;
    }
  if (!os->in_flight[slot]) return cudaSuccess;
  os->wait_done[slot] = true;
  return cudaStreamWaitEvent(st, os->selected[slot], 0);
}

// The votes of layer `c` are enqueued on c.st: selection on a side stream, gather on another.  While more score
// launches follow, two selections at a time (a selection takes one SM per segment, and a score launch whose CTAs wait
// for one another starts only when all of them fit beside what is running); `wide`: nothing follows, all side
// streams.  `scored_recorded`: the layer's event was recorded when its votes were launched (a deferred tail).
cudaError_t enqueue_tail(OverlapState* os, const PendingCall& c, bool beside_pipe, bool wide, int* launches,
                         bool scored_recorded = false) {
  const int slot = c.slot;
  const int si = wide ? slot % kSideStreams : slot % 2;
  cudaStream_t sel = os->side_select[si], gat = os->side_gather[si];
  if (g_prof_on == 1) sel = gat = c.st;  // timing of every kernel: one stream, so that the event pairs do not overlap
  cudaError_t e = scored_recorded ? cudaSuccess : cudaEventRecord(os->scored[slot], c.st);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(sel, os->scored[slot], 0);
  if (e == cudaSuccess && os->wait_done[slot]) e = cudaStreamWaitEvent(sel, os->done[slot], 0);
  os->wait_done[slot] = false;
  if (e != cudaSuccess) return e;
  e = launch_select_cta(c.pb, c.pooled_opt, c.budgets, c.offsets, c.kept_idx, c.capacity, c.status, sel, launches);
  if (e != cudaSuccess) return e;
  e = cudaEventRecord(os->selected[slot], sel);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(gat, os->selected[slot], 0);
  if (e != cudaSuccess) return e;
  // beside the two-layer score kernel an SM has registers left for one 128-thread gather CTA
  e = launch_gather(c.pb, c.offsets, c.kept_idx, c.k_out, c.v_out, c.capacity, gat, launches,
                    beside_pipe ? 128 : 256);
  if (e != cudaSuccess) return e;
  e = cudaEventRecord(os->done[slot], gat);
  if (e != cudaSuccess) return e;
  os->in_flight[slot] = true;
  return cudaSuccess;
}

// Selections and gathers that were held back until the score launch after theirs had gone out: the score kernel is
// then ahead of them in the order the device takes its work in and has its SMs first, and they fill the SMs it leaves.
cudaError_t flush_deferred(OverlapState* os, int* launches) {
  cudaError_t e = cudaSuccess;
  for (size_t i = 0; i < os->deferred.size() && e == cudaSuccess; ++i)
    e = enqueue_tail(os, os->deferred[i], true, true, launches, true);
  os->deferred.clear();
  return e;
}

// Launches the score kernel for the first n queued layers (pass 1) together with pass 2 of the pending layer and of
// all but the last of them -- of all of them when `finish` is set -- then the selections and gathers of the
// layers whose votes that gives.
cudaError_t launch_queue(OverlapState* os, int n, bool finish, int* launches) {
  if (n > (int)os->queue.size()) n = (int)os->queue.size();
  if (n == 0 && !(finish && os->pending.valid)) return cudaSuccess;
  if (n == 1 && finish && !os->pending.valid) {
    // a single layer and nothing to pair it with: both passes in the single-layer kernel
    const PendingCall& c = os->queue[0];
    cudaError_t e1 = launch_score_tensor(c.pb, c.cu_host.data(), c.status, c.pb.lse_opt ? 2 : 3, c.st, launches);
    if (e1 == cudaSuccess) e1 = flush_deferred(os, launches);
    if (e1 == cudaSuccess) e1 = enqueue_tail(os, c, false, true, launches);
    os->queue.clear();
    return e1;
  }
  const TcPlan* plans[kPipeMaxLayers];
  for (int i = 0; i < n; ++i) plans[i] = &os->queue[i].plan;
  cudaStream_t st = n > 0 ? os->queue[0].st : os->pending.st;
  // layers that came with their row statistics need the vote pass only (a queue holds one kind: see compress_impl)
  const bool votes_only = n > 0 && os->queue[0].pb.lse_opt != nullptr;
  const bool more_follow = !finish;                  // a full list went out because one more layer has come
  if (votes_only) finish = true;
  cudaError_t e = launch_score_pipe(os->pending.valid ? &os->pending.plan : nullptr, plans, n, finish, votes_only, st,
                                    launches);
  if (votes_only && more_follow) {
    // An ordinary launch takes the SMs that are free when it starts: selections that became ready at the same moment
    // would take a third of them for their 26 µs.  So this launch's selections and gathers are held back until the
    // next score launch is out (or a join), and the ones held back at the launch before go out now, behind this one.
    for (int i = 0; i < n && e == cudaSuccess; ++i) e = cudaEventRecord(os->scored[os->queue[i].slot], st);
    if (e == cudaSuccess) e = flush_deferred(os, launches);
    for (int i = 0; i < n && e == cudaSuccess; ++i) os->deferred.push_back(os->queue[i]);
    os->queue.erase(os->queue.begin(), os->queue.begin() + n);
    return e;
  }
  if (e == cudaSuccess) e = flush_deferred(os, launches);
  if (e == cudaSuccess && os->pending.valid) e = enqueue_tail(os, os->pending, true, finish, launches);
  os->pending.valid = false;
  const int n_voted = finish ? n : n - 1;
  for (int i = 0; i < n_voted && e == cudaSuccess; ++i) e = enqueue_tail(os, os->queue[i], true, finish, launches);
  if (!finish && n > 0) os->pending = os->queue[n - 1];
  os->queue.erase(os->queue.begin(), os->queue.begin() + n);
  return e;
}
cudaError_t flush_pending(OverlapState* os, int* launches) {
  cudaError_t e = cudaSuccess;
  while (!os->queue.empty() && (int)os->queue.size() > kPipeMaxLayers && e == cudaSuccess)
    e = launch_queue(os, kPipeMaxLayers, false, launches);
  if (e == cudaSuccess) e = launch_queue(os, (int)os->queue.size(), true, launches);
  if (e == cudaSuccess) e = flush_deferred(os, launches);
  return e;
}

// Calls on other streams whose workspace overlaps [ws, ws + bytes): their queued layers go out and `st` waits for what
// they have in flight, before a call on `st` carves that memory up for itself (g_overlap_mu held).
cudaError_t drain_states_sharing(const OverlapState* mine, const void* ws, size_t bytes, cudaStream_t st, int* launches) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  DeviceStates& d = g_overlap[dev];
  const char* lo = static_cast<const char*>(ws);
  for (int i = 0; i < kStatesPerDevice; ++i) {
    OverlapState& s = d.st[i];
    if (!d.used[i] || &s == mine || !s.sig.ws || state_idle(s)) continue;
    const char* olo = static_cast<const char*>(s.sig.ws);
    if (olo + s.sig.ws_bytes <= lo || lo + bytes <= olo) continue;
    e = flush_pending(&s, launches);
    for (int h = 0; h < kSlots && e == cudaSuccess; ++h)
      if (s.in_flight[h]) e = cudaStreamWaitEvent(st, s.done[h], 0);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// Makes `st` wait for every overlapped call still in flight on this device, whatever stream it was made on (no host
// wait).  Only the calls made on `st` itself are then forgotten: the others stay in flight for a join on their own
// stream, which still has to be ordered behind them.
cudaError_t join_overlapped(cudaStream_t st, int* launches) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaSuccess;
  std::lock_guard<std::mutex> lock(g_overlap_mu);
  DeviceStates& d = g_overlap[dev];
  for (int i = 0; i < kStatesPerDevice; ++i) {
    if (!d.used[i]) continue;
    OverlapState& s = d.st[i];
    e = flush_pending(&s, launches);
    if (e != cudaSuccess) return e;
    for (int h = 0; h < kSlots; ++h)
      if (s.in_flight[h]) {
        e = cudaStreamWaitEvent(st, s.done[h], 0);
        if (e != cudaSuccess) return e;
        if (d.owner[i] == st) s.in_flight[h] = false;
      }
  }
  return cudaSuccess;
}

int compress_impl(const slkv_params* p, const void* q_win, const void* k, const void* v, const int32_t* cu_dev,
                  const int32_t* cu_host, const int32_t* budgets, const float* lse_opt, void* k_out, void* v_out,
                  int64_t capacity,
                  int32_t* offsets, int32_t* kept_idx, float* pooled_opt, int32_t* status, void* ws,
                  size_t ws_bytes, cudaStream_t st, bool overlapped = false) {
  g_last_launches = 0;
  if (!q_win || !k || !v || !cu_dev || !budgets || !k_out || !v_out || !offsets || !kept_idx)
    return SLKV_ERR_NULL_PTR;
  Problem pb;
  int rc = describe(p, cu_host, &pb);
  if (rc != SLKV_OK) return rc;
  if (p->history_only) return SLKV_ERR_BAD_SHAPE;            // nothing to append behind the selected rows
  if (capacity < 0) return SLKV_ERR_CAPACITY;
  if (!aligned16(q_win) || !aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out))
    return SLKV_ERR_BAD_ALIGN;
  int path = 0;
  rc = resolve_path(pb, &path);
  if (rc != SLKV_OK) return rc;
  // pooling, offsets and selection run in one kernel when the segments fit it: one CTA per segment up to
  // 32768 history positions (overlapped calls), a thread-block cluster per segment otherwise
  const bool one_cta = overlapped && select_cta_supported(pb) && pb.tab.n_inline > 0;
  int launches = 0;
  if (!one_cta) {
    // ordinary call (or shapes the overlapped path does not take): everything on the caller's stream, after
    // whatever overlapped calls are still in flight
    cudaError_t je = join_overlapped(st, &launches);
    if (je != cudaSuccess) return cuda_fail(je);
    overlapped = false;
  }
  cudaError_t e = cudaSuccess;
  if (overlapped) {
    std::lock_guard<std::mutex> lock(g_overlap_mu);
    OverlapState* os = nullptr;
    e = overlap_state(st, &os, &launches);
    if (e != cudaSuccess) return cuda_fail(e);
    e = drain_states_sharing(os, ws, ws_bytes, st, &launches);
    if (e != cudaSuccess) return cuda_fail(e);
    ShapeSig sig;
    sig.ws = ws; sig.ws_bytes = ws_bytes; sig.n_seqs = pb.p.n_seqs; sig.n_kv_heads = pb.p.n_kv_heads; sig.R = pb.R;
    sig.max_hist = pb.max_hist; sig.path = path; sig.total_hist = pb.total_hist; sig.total_tokens = pb.total_tokens;
    if (!(sig == os->sig)) {
      // another shape or workspace: the carve-up changes, so nothing of the old one may still be in flight
      e = flush_pending(os, &launches);
      for (int h = 0; h < kSlots && e == cudaSuccess; ++h)
        if (os->in_flight[h]) {
          e = cudaStreamWaitEvent(st, os->done[h], 0);
          os->in_flight[h] = false;
        }
      if (e != cudaSuccess) return cuda_fail(e);
      os->sig = sig;
    }
    const int slot = (int)(os->seq % (unsigned)overlapped_slots(pb));
    rc = bind_workspace(&pb, ws, ws_bytes, path, true, slot);
    if (rc != SLKV_OK) return rc;
    ++os->seq;
    pb.cu = cu_dev; pb.q = q_win; pb.k = k; pb.v = v;
    pb.tab.cu_ptr = cu_dev;
    pb.lse_opt = lse_opt;
    // the score kernels leave a few SMs to the selection kernels of the layers before this one
    int sms = 148;
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int reserve = pb.n_seg < kSelectSmReserve ? pb.n_seg : kSelectSmReserve;
    pb.max_score_ctas = sms - reserve > 0 ? sms - reserve : 0;
    PendingCall cur;
    cur.valid = true; cur.pb = pb; cur.slot = slot; cur.budgets = budgets; cur.k_out = k_out; cur.v_out = v_out;
    cur.capacity = capacity; cur.offsets = offsets; cur.kept_idx = kept_idx; cur.pooled_opt = pooled_opt;
    cur.status = status; cur.st = st;
    cur.cu_host.assign(cu_host, cu_host + pb.p.n_seqs + 1);
    bool pipe = path == SLKV_PATH_TENSOR && score_pipe_supported(pb);
    if (pipe) {
      e = plan_score_tensor(pb, cu_host, status, &cur.plan);
      if (e != cudaSuccess) return cuda_fail(e);
      if (cur.plan.n_cta == 0) pipe = false;                        // no history: nothing to score
    }
    const bool queued = !os->queue.empty() || os->pending.valid;
    // a queue holds layers of one kind (both passes, or the vote pass alone) and of one stream
    const bool other_kind = os->pending.valid ? lse_opt != nullptr
                                              : (!os->queue.empty() && (os->queue[0].pb.lse_opt != nullptr) != (lse_opt != nullptr));
    if (queued && (!pipe || other_kind || (os->queue.empty() ? os->pending.st : os->queue[0].st) != st)) {
      e = flush_pending(os, &launches);
      if (e != cudaSuccess) return cuda_fail(e);
    }
    e = claim_slot(os, slot, st, &launches);
    if (e != cudaSuccess) return cuda_fail(e);
    if (pipe) {
      // Queue the layer; the score kernel takes a list of layers per launch (pass 1 of each beside pass 2 of the
      // one before) and goes out when the list is full and one more layer has come, or at a join.
      rc = enqueue_window_stats(pb, path, st, &launches);
      if (rc != SLKV_OK) return rc;
      os->queue.push_back(cur);
      if ((int)os->queue.size() > kPipeMaxLayers) {
        e = launch_queue(os, kPipeMaxLayers, false, &launches);
        if (e != cudaSuccess) return cuda_fail(e);
      }
    } else {
      rc = enqueue_votes(pb, path, cu_host, status, st, &launches);
      if (rc != SLKV_OK) return rc;
      e = enqueue_tail(os, cur, false, false, &launches);
      if (e != cudaSuccess) return cuda_fail(e);
    }
    g_last_launches = launches;
    return SLKV_OK;
  }
  rc = bind_workspace(&pb, ws, ws_bytes, path);
  if (rc != SLKV_OK) return rc;
  pb.cu = cu_dev; pb.q = q_win; pb.k = k; pb.v = v;
  pb.tab.cu_ptr = cu_dev;
  pb.lse_opt = lse_opt;
  const bool clustered = select_cluster_supported(pb);
  if (!clustered || pb.tab.n_inline == 0) {       // tables in global memory and / or the packed offsets
    e = launch_setup(pb, clustered ? nullptr : budgets, offsets, capacity, status, st, &launches);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  rc = enqueue_votes(pb, path, cu_host, status, st, &launches);
  if (rc != SLKV_OK) return rc;
  if (clustered) {
    // pooling, offsets and selection in one cluster kernel
    e = launch_select_cluster(pb, pooled_opt, budgets, offsets, kept_idx, capacity, status, st, &launches);
    if (e != cudaSuccess) return cuda_fail(e);
  } else {
    float* pooled = pooled_opt ? pooled_opt : pb.pooled_ws;
    e = launch_pool(pb, pooled, st, &launches);
    if (e != cudaSuccess) return cuda_fail(e);
    e = launch_select(pb, pooled, budgets, offsets, kept_idx, capacity, st, &launches);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  e = launch_gather(pb, offsets, kept_idx, k_out, v_out, capacity, st, &launches);
  if (e != cudaSuccess) return cuda_fail(e);
  g_last_launches = launches;
  return SLKV_OK;
}

}  // namespace

LaunchScope::LaunchScope(int kid, cudaStream_t st, int* launches) : kid_(kid), st_(st), slot_(-1) {
  ++*launches;
  if (!g_prof_on) return;
  const bool score_kid = kid == KID_SCORE_LSE || kid == KID_SCORE_VOTE || kid == KID_SCORE_FUSED || kid == KID_SCORE_PIPE;
  if (g_prof_on == 2 && !score_kid) return;
  if (!g_prof) g_prof = new std::vector<TimedLaunch>();
  TimedLaunch t{kid, prof_event(), prof_event()};
  if (!t.a || !t.b) return;
  cudaEventRecord(t.a, st);
  g_prof->push_back(t);
  slot_ = (int)g_prof->size() - 1;
}
LaunchScope::~LaunchScope() {
  if (slot_ >= 0) cudaEventRecord((*g_prof)[slot_].b, st_);
}

}  // namespace slkv

using namespace slkv;

extern "C" {

const char* slkv_strerror(int status) {
  switch (status) {
    case SLKV_OK: return "SLKV_OK";
    case SLKV_ERR_NULL_PTR: return "SLKV_ERR_NULL_PTR: a required pointer is NULL";
    case SLKV_ERR_BAD_SHAPE: return "SLKV_ERR_BAD_SHAPE: size, count or stride out of range";
    case SLKV_ERR_BAD_DTYPE: return "SLKV_ERR_BAD_DTYPE: unknown or unsupported dtype / mode / path";
    case SLKV_ERR_BAD_ALIGN: return "SLKV_ERR_BAD_ALIGN: pointer or stride not 16-byte aligned";
    case SLKV_ERR_BUDGET_SUM: return "SLKV_ERR_BUDGET_SUM: total smaller than heads * fixed";
    case SLKV_ERR_NEG_INF_SC: return "SLKV_ERR_NEG_INF_SC: INF_sc negative or not finite";
    case SLKV_ERR_CAPACITY: return "SLKV_ERR_CAPACITY: packed output capacity too small";
    case SLKV_ERR_WORKSPACE: return "SLKV_ERR_WORKSPACE: workspace missing or too small";
    case SLKV_ERR_CUDA: return "SLKV_ERR_CUDA: a CUDA runtime call failed";
    case SLKV_ERR_DEVICE_TIMEOUT: return "SLKV_ERR_DEVICE_TIMEOUT: a bounded device-side wait ran out";
    default: return "unknown slkv status";
  }
}

int slkv_profile_enable(int on) {
  g_prof_on = on < 0 ? 0 : (on > 2 ? 1 : on);
  return SLKV_OK;
}

int slkv_profile_collect(float* total_ms, int32_t* launches, int32_t n_kernels) {
  if (!total_ms || !launches) return SLKV_ERR_NULL_PTR;
  for (int i = 0; i < n_kernels; ++i) { total_ms[i] = 0.f; launches[i] = 0; }
  if (!g_prof) return SLKV_OK;
  if (!g_prof_free) g_prof_free = new std::vector<cudaEvent_t>();
  int rc = SLKV_OK;
  for (TimedLaunch& t : *g_prof) {
    float ms = 0.f;
    cudaError_t e = cudaEventSynchronize(t.b);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, t.a, t.b);
    if (e != cudaSuccess) rc = cuda_fail(e);
    else if (t.kid < n_kernels) { total_ms[t.kid] += ms; launches[t.kid] += 1; }
    g_prof_free->push_back(t.a);
    g_prof_free->push_back(t.b);
  }
  g_prof->clear();
  return rc;
}

const char* slkv_kernel_name(int kernel_id) {
  static const char* names[KID_COUNT] = {"k_setup", "k_score_lse", "k_score_vote", "k_pool", "k_select",
                                         "k_gather", "k_alloc", "k_score_fused", "k_score_pipe", "k_window_stats",
                                         "k_merge_lse", "k_behavior", "k_cp"};
  return (kernel_id >= 0 && kernel_id < KID_COUNT) ? names[kernel_id] : "";
}

int slkv_kernel_count(void) { return KID_COUNT; }

int slkv_trace_set_buffer(void* dev_buf, size_t bytes) {
  set_tensor_trace(dev_buf, dev_buf ? bytes : 0);
  return SLKV_OK;
}

int slkv_last_cuda_error(void) { return g_last_cuda_error; }
int slkv_last_launch_count(void) { return g_last_launches; }
int slkv_version(void) { return 300; }

int slkv_debug_expire_next_wait(int on) {
  expire_next_wait(on != 0);
  return SLKV_OK;
}

int slkv_behavior_scores(const float* attn, int64_t n_rows, int32_t row_len, int64_t row_stride,
                         const int32_t* needle_idx, int32_t n_needle, int64_t needle_stride, const int32_t* topk_idx,
                         int32_t n_topk, int64_t topk_stride, float* sf_sc, float* lg_sc, float* inf_sc, void* stream) {
  if (!attn || !needle_idx || !topk_idx || !sf_sc || !lg_sc || !inf_sc) return SLKV_ERR_NULL_PTR;
  if (n_rows < 0 || n_rows > (1ll << 34) || row_len < 1 || row_stride < 0 || n_needle < 0 || n_needle > 4096 ||
      n_topk < 0 || n_topk > 4096 || needle_stride < 0 || topk_stride < 0)
    return SLKV_ERR_BAD_SHAPE;
  cudaError_t e = launch_behavior(attn, row_stride, row_len, n_rows, needle_idx, n_needle, needle_stride, topk_idx,
                                  n_topk, topk_stride, sf_sc, lg_sc, inf_sc, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e);
  return SLKV_OK;
}

// ---- context-parallel selection (slkv_cp.cu) -----------------------------------------------------------------
int slkv_cp_merge_lse(const slkv_params* p, const float* lse_parts, int32_t n_parts, float* lse_out, void* stream) {
  if (!p || !lse_parts || !lse_out) return SLKV_ERR_NULL_PTR;
  if (n_parts < 1 || n_parts > 4096 || p->n_seqs != 1 || p->n_q_heads < 1 || p->window < 1 || p->window > kMaxWindow)
    return SLKV_ERR_BAD_SHAPE;
  if (p->lse_units != SLKV_LSE_LN && p->lse_units != SLKV_LSE_LOG2) return SLKV_ERR_BAD_DTYPE;
  int launches = 0;
  const float to_log2 = p->lse_units == SLKV_LSE_LOG2 ? 1.0f : 1.4426950408889634f;
  cudaError_t e = launch_cp_merge_lse(lse_parts, n_parts, (long long)p->n_q_heads * p->window, to_log2, lse_out,
                                      (cudaStream_t)stream, &launches);
  return e == cudaSuccess ? SLKV_OK : cuda_fail(e);
}

int slkv_cp_select_init(const int32_t* budgets, int32_t n_kv_heads, int32_t window, int64_t seq_len, uint32_t* prefix,
                        int32_t* need, void* stream) {
  if (!budgets || !prefix || !need) return SLKV_ERR_NULL_PTR;
  if (n_kv_heads < 1 || n_kv_heads > 65535 || window < 1 || window > kMaxWindow || seq_len < 0 || seq_len >= (1ll << 31))
    return SLKV_ERR_BAD_SHAPE;
  int launches = 0;
  cudaError_t e = launch_cp_need_init(budgets, n_kv_heads, window, seq_len, prefix, need, (cudaStream_t)stream, &launches);
  return e == cudaSuccess ? SLKV_OK : cuda_fail(e);
}

int slkv_cp_histogram(const float* pooled, int32_t n_kv_heads, int64_t row_stride, int32_t own_begin, int32_t own_count,
                      int32_t level, const uint32_t* prefix, int32_t* hist, void* stream) {
  if (!pooled || !prefix || !hist) return SLKV_ERR_NULL_PTR;
  if (n_kv_heads < 1 || n_kv_heads > 65535 || row_stride < 0 || own_begin < 0 || own_count < 0 ||
      (int64_t)own_begin + own_count > row_stride || level < 0 || level > 2)
    return SLKV_ERR_BAD_SHAPE;
  int launches = 0;
  cudaError_t e = launch_cp_histogram(pooled, n_kv_heads, row_stride, own_begin, own_count, level, prefix, hist,
                                      (cudaStream_t)stream, &launches);
  return e == cudaSuccess ? SLKV_OK : cuda_fail(e);
}

int slkv_cp_descend(const int32_t* hist, int32_t n_kv_heads, int32_t level, uint32_t* prefix, int32_t* need,
                    void* stream) {
  if (!hist || !prefix || !need) return SLKV_ERR_NULL_PTR;
  if (n_kv_heads < 1 || n_kv_heads > 65535 || level < 0 || level > 2) return SLKV_ERR_BAD_SHAPE;
  int launches = 0;
  cudaError_t e = launch_cp_descend(hist, n_kv_heads, level, prefix, need, (cudaStream_t)stream, &launches);
  return e == cudaSuccess ? SLKV_OK : cuda_fail(e);
}

int slkv_cp_local_ties(const int32_t* hist_local, const uint32_t* prefix, int32_t n_kv_heads, int32_t* ties,
                       void* stream) {
  if (!hist_local || !prefix || !ties) return SLKV_ERR_NULL_PTR;
  if (n_kv_heads < 1 || n_kv_heads > 65535) return SLKV_ERR_BAD_SHAPE;
  int launches = 0;
  cudaError_t e = launch_cp_local_ties(hist_local, prefix, n_kv_heads, ties, (cudaStream_t)stream, &launches);
  return e == cudaSuccess ? SLKV_OK : cuda_fail(e);
}

size_t slkv_cp_workspace_bytes(int32_t n_kv_heads, int32_t own_count, int64_t out_capacity_rows) {
  if (n_kv_heads < 1 || own_count < 0 || out_capacity_rows < 0) return 0;
  // source rows of the packed rows; rows and tie shares per head; two counts per slice of the owned range and head
  const size_t slices = (size_t)cp_slices(own_count) * (size_t)n_kv_heads;
  return align_up((size_t)out_capacity_rows * sizeof(int32_t)) + 2 * align_up((size_t)n_kv_heads * sizeof(int32_t)) +
         2 * align_up(slices * sizeof(int32_t));
}

int slkv_cp_emit(const slkv_params* p, const void* k, const void* v, int64_t rows, const float* pooled,
                 int64_t row_stride, int32_t own_begin, int32_t own_count, int64_t pos0, const uint32_t* threshold,
                 const int32_t* need, const int32_t* ties_all, int32_t n_parts, int32_t part, int32_t window_rows,
                 int64_t window_pos0, void* k_out, void* v_out, int64_t out_capacity_rows, int32_t* offsets,
                 int32_t* kept_idx, int32_t* status, void* workspace, size_t workspace_bytes, void* stream) {
  g_last_launches = 0;
  if (!p || !k || !v || !pooled || !threshold || !need || !ties_all || !k_out || !v_out || !offsets || !kept_idx)
    return SLKV_ERR_NULL_PTR;
  const int32_t cu1[2] = {0, (int32_t)(rows < (1ll << 31) && rows >= 0 ? rows : -1)};
  Problem pb;
  int rc = describe(p, cu1, &pb);                    // validates dtype, head counts, strides
  if (rc != SLKV_OK) return rc;
  if (n_parts < 1 || part < 0 || part >= n_parts || window_rows < 0 || window_rows > p->window || window_rows > rows ||
      own_begin < 0 || own_count < 0 || (int64_t)own_begin + own_count > rows - window_rows ||
      (int64_t)own_begin + own_count > row_stride || pos0 < 0 || pos0 + own_count >= (1ll << 31) || window_pos0 < 0 ||
      window_pos0 + window_rows >= (1ll << 31))
    return SLKV_ERR_BAD_SHAPE;
  if (out_capacity_rows < 0) return SLKV_ERR_CAPACITY;
  if (!aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out)) return SLKV_ERR_BAD_ALIGN;
  const size_t need_ws = slkv_cp_workspace_bytes(p->n_kv_heads, own_count, out_capacity_rows);
  if (!workspace || workspace_bytes < need_ws || reinterpret_cast<uintptr_t>(workspace) % kAlign != 0)
    return SLKV_ERR_WORKSPACE;
  char* w = static_cast<char*>(workspace);
  int32_t* gather_src = reinterpret_cast<int32_t*>(w);
  int32_t* rows_h = reinterpret_cast<int32_t*>(w + align_up((size_t)out_capacity_rows * sizeof(int32_t)));
  int32_t* take_h = rows_h + align_up((size_t)p->n_kv_heads * sizeof(int32_t)) / sizeof(int32_t);
  int32_t* cnt_gt = take_h + align_up((size_t)p->n_kv_heads * sizeof(int32_t)) / sizeof(int32_t);
  int32_t* cnt_eq = cnt_gt + align_up((size_t)cp_slices(own_count) * p->n_kv_heads * sizeof(int32_t)) / sizeof(int32_t);
  cudaStream_t st = (cudaStream_t)stream;
  int launches = 0;
  cudaError_t e = launch_cp_emit(pooled, row_stride, own_begin, own_count, pos0, threshold, need, ties_all,
                                 p->n_kv_heads, part, window_rows, rows - window_rows, window_pos0, out_capacity_rows,
                                 offsets, kept_idx, gather_src, rows_h, take_h, cnt_gt, cnt_eq, status, st, &launches);
  if (e != cudaSuccess) return cuda_fail(e);
  pb.total_tokens = rows;
  pb.n_seg = p->n_kv_heads;
  pb.k = k; pb.v = v;
  pb.gather_src = gather_src;
  e = launch_gather(pb, offsets, kept_idx, k_out, v_out, out_capacity_rows, st, &launches, 256);
  if (e != cudaSuccess) return cuda_fail(e);
  g_last_launches = launches;
  return SLKV_OK;
}

int slkv_alloc_budgets_ex(const float* inf_sc, int32_t n_layers, int32_t n_heads, int32_t fixed, int64_t total,
                          const slkv_alloc_options* opt, int32_t* budgets, int32_t* status, void* stream) {
  if (!inf_sc || !budgets) return SLKV_ERR_NULL_PTR;
  if (n_layers < 1 || n_heads < 1 || n_layers > 1024 || (int64_t)n_layers * n_heads > 16384)
    return SLKV_ERR_BAD_SHAPE;
  const int64_t n = (int64_t)n_layers * n_heads;
  if (fixed < 0 || total < n * fixed) return SLKV_ERR_BUDGET_SUM;
  if (total > 0x7fffffffll) return SLKV_ERR_BAD_SHAPE;
  int within = 0, paper = 0;
  long long cap = -1;
  if (opt) {
    if (opt->head_normaliser != SLKV_NORM_GLOBAL && opt->head_normaliser != SLKV_NORM_WITHIN_LAYER) return SLKV_ERR_BAD_DTYPE;
    if (opt->rounding != SLKV_ROUND_SUM_EXACT && opt->rounding != SLKV_ROUND_PAPER) return SLKV_ERR_BAD_DTYPE;
    if (opt->cap < 0 || opt->cap > 0x7fffffffll) return SLKV_ERR_BAD_SHAPE;
    within = opt->head_normaliser == SLKV_NORM_WITHIN_LAYER;
    paper = opt->rounding == SLKV_ROUND_PAPER;
    if (opt->cap > 0) {
      cap = opt->cap;
      // a cap below the fixed part, or a total that does not fit under the cap (where the total is to be met)
      if (cap < fixed || (!paper && total > n * cap)) return SLKV_ERR_BUDGET_SUM;
    }
  }
  cudaError_t e = launch_alloc(inf_sc, n_layers, n_heads, fixed, total, within, paper, cap, budgets, status,
                               (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e);
  return SLKV_OK;
}

int slkv_alloc_budgets(const float* inf_sc, int32_t n_layers, int32_t n_heads, int32_t fixed, int64_t total,
                       int32_t* budgets, int32_t* status, void* stream) {
  return slkv_alloc_budgets_ex(inf_sc, n_layers, n_heads, fixed, total, nullptr, budgets, status, stream);
}

size_t slkv_workspace_bytes(const slkv_params* p, const int32_t* cu_seqlens_host) {
  Problem pb;
  if (describe(p, cu_seqlens_host, &pb) != SLKV_OK) return 0;
  return layout_of(pb).total;
}

size_t slkv_workspace_bytes_overlapped(const slkv_params* p, const int32_t* cu_seqlens_host) {
  Problem pb;
  if (describe(p, cu_seqlens_host, &pb) != SLKV_OK) return 0;
  return layout_of(pb, true).total;
}

int slkv_compress_overlapped(const slkv_params* p, const void* q_win, const void* k, const void* v,
                             const int32_t* cu_seqlens_dev, const int32_t* cu_seqlens_host, const int32_t* budgets,
                             const float* lse_opt, void* k_out, void* v_out, int64_t out_capacity_rows,
                             int32_t* offsets, int32_t* kept_idx, float* pooled_opt, int32_t* status, void* workspace,
                             size_t workspace_bytes, void* stream) {
  {
    Problem pb;                                   // the overlapped layout is the larger one: check it up front
    if (p && cu_seqlens_host && describe(p, cu_seqlens_host, &pb) == SLKV_OK && workspace &&
        workspace_bytes < layout_of(pb, true).total)
      return SLKV_ERR_WORKSPACE;
  }
  return compress_impl(p, q_win, k, v, cu_seqlens_dev, cu_seqlens_host, budgets, lse_opt, k_out, v_out,
                       out_capacity_rows, offsets, kept_idx, pooled_opt, status, workspace, workspace_bytes,
                       (cudaStream_t)stream, true);
}

int slkv_join(void* stream) {
  int launches = 0;
  cudaError_t e = join_overlapped((cudaStream_t)stream, &launches);
  g_last_launches = launches;
  if (e != cudaSuccess) return cuda_fail(e);
  return SLKV_OK;
}

int64_t slkv_pooled_elems(const slkv_params* p, const int32_t* cu_seqlens_host) {
  Problem pb;
  if (describe(p, cu_seqlens_host, &pb) != SLKV_OK) return -1;
  return (int64_t)pb.p.n_kv_heads * pb.total_hist;
}

int64_t slkv_packed_rows_upper_bound(const slkv_params* p, const int32_t* cu_seqlens_host) {
  Problem pb;
  if (describe(p, cu_seqlens_host, &pb) != SLKV_OK) return -1;
  return (int64_t)pb.p.n_kv_heads * pb.total_tokens;
}

namespace {
// slkv_score and slkv_row_lse: the votes pooled into `pooled`, or the rows' log-sum-exp into `lse_out`.
int score_impl(const slkv_params* p, const void* q_win, const void* k, const int32_t* cu_seqlens_dev,
               const int32_t* cu_seqlens_host, const float* lse_opt, float* pooled, float* lse_out, int32_t* status,
               void* workspace, size_t workspace_bytes, void* stream) {
  g_last_launches = 0;
  if (!q_win || !k || !cu_seqlens_dev || (!pooled && !lse_out)) return SLKV_ERR_NULL_PTR;
  Problem pb;
  int rc = describe(p, cu_seqlens_host, &pb);
  if (rc != SLKV_OK) return rc;
  if (!aligned16(q_win) || !aligned16(k)) return SLKV_ERR_BAD_ALIGN;
  int path = 0;
  rc = resolve_path(pb, &path);
  if (rc != SLKV_OK) return rc;
  rc = bind_workspace(&pb, workspace, workspace_bytes, path);
  if (rc != SLKV_OK) return rc;
  pb.cu = cu_seqlens_dev; pb.q = q_win; pb.k = k; pb.v = nullptr;
  pb.tab.cu_ptr = cu_seqlens_dev;
  pb.lse_opt = lse_opt;
  if (p->history_only) cu_seqlens_host = pb.cu_virtual;      // one sequence: the tables are inline, cu_seqlens_dev unread
  cudaStream_t st = (cudaStream_t)stream;
  int launches = 0;
  cudaError_t e = join_overlapped(st, &launches);  // the workspace may still serve an overlapped call
  if (e != cudaSuccess) return cuda_fail(e);
  if (pb.tab.n_inline == 0) {
    e = launch_setup(pb, nullptr, nullptr, 0, nullptr, st, &launches);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  if (lse_out) {
    // row statistics only: pass 1, the window keys' share where the domain has one, then the merge
    rc = enqueue_window_stats(pb, path, st, &launches);
    if (rc != SLKV_OK) return rc;
    e = path == SLKV_PATH_TENSOR ? launch_score_tensor(pb, cu_seqlens_host, status, 1, st, &launches)
                                 : launch_score_simt(pb, 1, st, &launches);
    if (e == cudaSuccess)
      e = path == SLKV_PATH_TENSOR ? launch_merge_lse_tensor(pb, cu_seqlens_host, lse_out, st, &launches)
                                   : launch_merge_lse_simt(pb, lse_out, st, &launches);
    if (e != cudaSuccess) return cuda_fail(e);
    g_last_launches = launches;
    return SLKV_OK;
  }
  rc = enqueue_votes(pb, path, cu_seqlens_host, status, st, &launches);
  if (rc != SLKV_OK) return rc;
  e = launch_pool(pb, pooled, st, &launches);
  if (e != cudaSuccess) return cuda_fail(e);
  g_last_launches = launches;
  return SLKV_OK;
}
}  // namespace

int slkv_score(const slkv_params* p, const void* q_win, const void* k, const int32_t* cu_seqlens_dev,
               const int32_t* cu_seqlens_host, const float* lse_opt, float* pooled, int32_t* status, void* workspace,
               size_t workspace_bytes, void* stream) {
  if (!pooled) return SLKV_ERR_NULL_PTR;
  return score_impl(p, q_win, k, cu_seqlens_dev, cu_seqlens_host, lse_opt, pooled, nullptr, status, workspace,
                    workspace_bytes, stream);
}

int slkv_row_lse(const slkv_params* p, const void* q_win, const void* k, const int32_t* cu_seqlens_dev,
                 const int32_t* cu_seqlens_host, float* lse_out, int32_t* status, void* workspace,
                 size_t workspace_bytes, void* stream) {
  if (!lse_out) return SLKV_ERR_NULL_PTR;
  return score_impl(p, q_win, k, cu_seqlens_dev, cu_seqlens_host, nullptr, nullptr, lse_out, status, workspace,
                    workspace_bytes, stream);
}

}  // extern "C"

// Host-side validation of slkv_score's arguments without a workspace (for entry points that bring their own).
int slkv::check_score_args(const slkv_params* p, const void* q_win, const void* k, const int32_t* cu_seqlens_dev,
                           const int32_t* cu_seqlens_host, const float* pooled) {
  if (!q_win || !k || !cu_seqlens_dev || !pooled) return SLKV_ERR_NULL_PTR;
  Problem pb;
  int rc = describe(p, cu_seqlens_host, &pb);
  if (rc != SLKV_OK) return rc;
  if (!aligned16(q_win) || !aligned16(k)) return SLKV_ERR_BAD_ALIGN;
  int path = 0;
  return resolve_path(pb, &path);
}

extern "C" {

int slkv_compress(const slkv_params* p, const void* q_win, const void* k, const void* v,
                  const int32_t* cu_seqlens_dev, const int32_t* cu_seqlens_host, const int32_t* budgets,
                  const float* lse_opt, void* k_out, void* v_out, int64_t out_capacity_rows, int32_t* offsets,
                  int32_t* kept_idx, float* pooled_opt, int32_t* status, void* workspace, size_t workspace_bytes,
                  void* stream) {
  return compress_impl(p, q_win, k, v, cu_seqlens_dev, cu_seqlens_host, budgets, lse_opt, k_out, v_out,
                       out_capacity_rows, offsets, kept_idx, pooled_opt, status, workspace, workspace_bytes,
                       (cudaStream_t)stream);
}

// ---- host-buffer variant ---------------------------------------------------------------------------
namespace {
struct HostArena {
  size_t q, k, v, cu, budgets, k_out, v_out, offsets, kept, status, ws, total;
};
bool host_arena_layout(const Problem& pb, int64_t capacity, HostArena* A) {
  const slkv_params& p = pb.p;
  const size_t e = pb.elem, d = p.head_dim;
  size_t o = 0;
  A->q = o; o = align_up(o + (size_t)p.n_seqs * p.window * p.n_q_heads * d * e);
  A->k = o; o = align_up(o + (size_t)pb.total_tokens * p.n_kv_heads * d * e);
  A->v = o; o = align_up(o + (size_t)pb.total_tokens * p.n_kv_heads * d * e);
  A->cu = o; o = align_up(o + (size_t)(p.n_seqs + 1) * 4);
  A->budgets = o; o = align_up(o + (size_t)p.n_kv_heads * 4);
  A->k_out = o; o = align_up(o + (size_t)capacity * d * e);
  A->v_out = o; o = align_up(o + (size_t)capacity * d * e);
  A->offsets = o; o = align_up(o + (size_t)(pb.n_seg + 1) * 4);
  A->kept = o; o = align_up(o + (size_t)capacity * 4);
  A->status = o; o = align_up(o + 4);
  A->ws = o; o = align_up(o + layout_of(pb).total);
  A->total = o;
  return true;
}
bool dense_strides(const slkv_params& p) {
  const int64_t d = p.head_dim;
  return p.k_stride_head == d && p.k_stride_tok == d * p.n_kv_heads && p.v_stride_head == d &&
         p.v_stride_tok == d * p.n_kv_heads && p.q_stride_head == d && p.q_stride_row == d * p.n_q_heads &&
         p.q_stride_seq == d * p.n_q_heads * p.window;
}
}  // namespace

size_t slkv_compress_host_arena_bytes(const slkv_params* p, const int32_t* cu_seqlens_host,
                                      int64_t out_capacity_rows) {
  Problem pb;
  if (describe(p, cu_seqlens_host, &pb) != SLKV_OK || out_capacity_rows < 0) return 0;
  HostArena A;
  host_arena_layout(pb, out_capacity_rows, &A);
  return A.total;
}

int slkv_compress_host(const slkv_params* p, const void* q_win, const void* k, const void* v,
                       const int32_t* cu_seqlens_host, const int32_t* budgets, void* k_out, void* v_out,
                       int64_t out_capacity_rows, int32_t* offsets, int32_t* kept_idx, int64_t* rows_out,
                       void* arena, size_t arena_bytes, void* stream) {
  g_last_launches = 0;
  if (!q_win || !k || !v || !budgets || !k_out || !v_out || !offsets || !kept_idx || !arena)
    return SLKV_ERR_NULL_PTR;
  Problem pb;
  int rc = describe(p, cu_seqlens_host, &pb);
  if (rc != SLKV_OK) return rc;
  if (!dense_strides(*p) || p->history_only) return SLKV_ERR_BAD_SHAPE;
  if (out_capacity_rows < 0) return SLKV_ERR_CAPACITY;
  if (reinterpret_cast<uintptr_t>(arena) % kAlign != 0) return SLKV_ERR_BAD_ALIGN;
  HostArena A;
  host_arena_layout(pb, out_capacity_rows, &A);
  if (arena_bytes < A.total) return SLKV_ERR_WORKSPACE;
  // rows that will be written, known on the host because the budgets are (Algorithm 3 l.1-4, l.7)
  int64_t rows = 0;
  for (int s = 0; s < p->n_seqs; ++s) {
    const int64_t len = cu_seqlens_host[s + 1] - cu_seqlens_host[s];
    for (int h = 0; h < p->n_kv_heads; ++h) {
      int64_t c = budgets[h] > p->window ? budgets[h] : p->window;
      rows += len < c ? len : c;
    }
  }
  if (rows_out) *rows_out = rows;
  if (rows > out_capacity_rows) return SLKV_ERR_CAPACITY;

  cudaStream_t st = (cudaStream_t)stream;
  unsigned char* b = static_cast<unsigned char*>(arena);
  const size_t e = pb.elem, d = p->head_dim;
  cudaError_t ce;
#define SLKV_CP(dst, src, n, kind)                                  \
  do {                                                              \
    if ((n) > 0) {                                                  \
      ce = cudaMemcpyAsync((dst), (src), (n), (kind), st);          \
      if (ce != cudaSuccess) return cuda_fail(ce);                  \
    }                                                               \
  } while (0)
  SLKV_CP(b + A.q, q_win, (size_t)p->n_seqs * p->window * p->n_q_heads * d * e, cudaMemcpyHostToDevice);
  SLKV_CP(b + A.k, k, (size_t)pb.total_tokens * p->n_kv_heads * d * e, cudaMemcpyHostToDevice);
  SLKV_CP(b + A.v, v, (size_t)pb.total_tokens * p->n_kv_heads * d * e, cudaMemcpyHostToDevice);
  SLKV_CP(b + A.cu, cu_seqlens_host, (size_t)(p->n_seqs + 1) * 4, cudaMemcpyHostToDevice);
  SLKV_CP(b + A.budgets, budgets, (size_t)p->n_kv_heads * 4, cudaMemcpyHostToDevice);
  rc = compress_impl(p, b + A.q, b + A.k, b + A.v, reinterpret_cast<int32_t*>(b + A.cu), cu_seqlens_host,
                     reinterpret_cast<int32_t*>(b + A.budgets), nullptr, b + A.k_out, b + A.v_out, out_capacity_rows,
                     reinterpret_cast<int32_t*>(b + A.offsets), reinterpret_cast<int32_t*>(b + A.kept), nullptr,
                     nullptr, b + A.ws, arena_bytes - A.ws, st);
  if (rc != SLKV_OK) return rc;
  SLKV_CP(offsets, b + A.offsets, (size_t)(pb.n_seg + 1) * 4, cudaMemcpyDeviceToHost);
  SLKV_CP(kept_idx, b + A.kept, (size_t)rows * 4, cudaMemcpyDeviceToHost);
  SLKV_CP(k_out, b + A.k_out, (size_t)rows * d * e, cudaMemcpyDeviceToHost);
  SLKV_CP(v_out, b + A.v_out, (size_t)rows * d * e, cudaMemcpyDeviceToHost);
#undef SLKV_CP
  ce = cudaStreamSynchronize(st);
  if (ce != cudaSuccess) return cuda_fail(ce);
  return SLKV_OK;
}

}  // extern "C"
