// Host side of the C ABI declared in include/fltop.h: argument validation,
// workspace carve-up and kernel launches on the caller's stream.
#include <algorithm>
#include <cmath>
#include <limits>
#include <new>

#include "../../include/fltop.h"
#include "fltop_internal.h"

using namespace fltop;

namespace {
constexpr int kIoMaxGroups = 16;
constexpr int kIoStreams = kIoMaxGroups;  // a stream per group: the groups' kernels run side by side
constexpr int kIoGroupSize = 8;  // utterances per group (more when B > 8 * kIoMaxGroups)

// Staging of fltop_decode_host: device copies of the inputs and outputs, pinned host mirrors of
// the small outputs, the streams and events of the copy / decode pipeline.
struct HostIo {
  bool ready = false;
  unsigned char* dev = nullptr;      // one device allocation
  unsigned char* pinned = nullptr;   // one pinned host allocation
  unsigned char* d_logp = nullptr;   // [max_batch, max_frames, V] elements of emission_dtype
  int32_t* d_lengths = nullptr;      // [max_batch]
  int32_t* d_tokens = nullptr;       // [max_batch, K, L]
  // lens [n,K], scores [n,K], nhyp [n], status [n] of a group of n utterances lie back to back
  // (2K + 2 words per utterance), so that one copy brings a group's small outputs home
  int32_t* d_small = nullptr;        // [max_batch * (2K + 2)]
  int32_t* p_small = nullptr;        // pinned host mirror
  int32_t* p_lengths = nullptr;      // pinned, [max_batch], in slot order
  int32_t* order = nullptr;          // [max_batch] pageable host scratch
  cudaStream_t stream[kIoStreams] = {};
  cudaEvent_t begin = nullptr, end[kIoStreams] = {}, done[kIoMaxGroups] = {};
  int64_t h2d_bytes = 0, d2h_bytes = 0;  // of the most recent call
};
}  // namespace

struct fltop_handle {
  fltop_config cfg;
  HostIo io;
  float log_r;
  bool owns_workspace;
  unsigned char* ws;
  size_t ws_bytes;
  // regions of the workspace
  int32_t* counts;        // survivor region (null until a call needs it)
  Survivor* entries;
  unsigned char* survivor_extra;  // the region when the library allocated it by itself
  size_t survivor_bytes, counts_bytes;
  TrieNode* nodes;
  int32_t* state;
  int32_t* stats;
  int32_t* prune_error;   // device word: a bulk copy of the prune kernel did not complete in time
  int32_t last_B, last_T;
  bool last_fused;        // the most recent call pruned inside the decode kernel
  cudaStream_t last_stream;
  int64_t frame_cap;      // frames per utterance the survivor buffers hold
  int64_t nodes_per_utt;
  size_t beam_state_bytes;
  int last_cuda;
  int64_t launches;
  int32_t block_threads;  // 0 = chosen by the library
  int32_t fusion;         // 1 = the decode kernel prunes where it can
  int32_t warp_mode;      // warp-per-utterance kernel: 0 never, 1 when it pays, 2 whenever it can
  int32_t rows_mode;      // 1: character vocabularies with beams up to 64 take the row kernel
  bool profiling;
  bool prof_valid;
  cudaEvent_t ev[3];
  // instrumented launches (fltop_set_test_hook); all off by default
  uint32_t* hook_masks;
  long long* hook_clocks;
  int32_t hook_frame0, hook_frames, hook_table_slots, hook_prune_staged;
};

namespace {

constexpr size_t kMaxSmem = 227 * 1024;
constexpr size_t kAlign = 256;

size_t up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

bool config_ok(const fltop_config* c) {
  if (!c) return false;
  if (c->vocab_size < 2 || c->vocab_size > 8192) return false;
  if (c->blank_id < 0 || c->blank_id >= c->vocab_size) return false;
  if (c->beam_width < 1 || c->beam_width > 2048) return false;
  if (!(c->threshold_r >= 0.f && c->threshold_r <= 1.f)) return false;  // rejects NaN too
  if (c->max_batch < 1 || c->max_frames < 1 || c->max_out_len < 1) return false;
  if (c->max_chunk_frames < 0 || c->max_chunk_frames > c->max_frames) return false;
  if (c->top_n < 0) return false;
  if (c->beam_threshold != c->beam_threshold) return false;  // NaN
  if (c->merge_max != 0 && c->merge_max != 1) return false;
  if (c->emission_dtype < FLTOP_EMISSION_F32 || c->emission_dtype > FLTOP_EMISSION_BF16) return false;
  if (c->max_trie_nodes < 0) return false;
  if (c->device < 0) return false;
  if ((int64_t)(c->beam_width + 1) * c->max_frames + 2 > (int64_t)std::numeric_limits<int32_t>::max())
    return false;
  if (decode_smem_bytes(c->beam_width, c->vocab_size) > kMaxSmem) return false;
  if (c->workspace && (reinterpret_cast<uintptr_t>(c->workspace) % kAlign) != 0) return false;
  return true;
}

struct Layout {
  size_t survivors, nodes, state, stats, flags, total, beam_state;
  size_t survivor_bytes, counts_bytes;  // the survivor region: counts, then entries
  bool survivors_inside;                // the region is part of the workspace
  int64_t frame_cap, nodes_per_utt;
};

// A vocabulary that the decode kernels cannot prune themselves always needs survivor lists
// (narrower ones get them on the first call that cannot be pruned inside, if ever).
bool needs_survivor_lists(const fltop_config& c) { return c.vocab_size > 1024; }

Layout layout_of(const fltop_config& c) {
  Layout l;
  l.frame_cap = c.max_chunk_frames > 0 ? c.max_chunk_frames : c.max_frames;
  // a frame creates at most beam_width nodes, handed out in even-sized runs; ids 0 and 1 are fixed
  const int64_t worst = (int64_t)((c.beam_width + 1) & ~1) * c.max_frames + 2;
  int64_t cap = worst;
  if (c.max_trie_nodes > 0) {
    cap = std::min<int64_t>(worst, std::max<int64_t>(c.max_trie_nodes, 2 * c.beam_width + 4));
    cap = (cap + 1) & ~(int64_t)1;
  }
  l.nodes_per_utt = cap;
  const size_t frames = (size_t)c.max_batch * (size_t)l.frame_cap;
  l.counts_bytes = up(frames * sizeof(int32_t));
  l.survivor_bytes = l.counts_bytes + up(frames * (size_t)c.vocab_size * sizeof(Survivor));
  l.survivors_inside = needs_survivor_lists(c);
  size_t off = 0;
  l.survivors = off;
  if (l.survivors_inside) off += l.survivor_bytes;
  l.nodes = off; off += up((size_t)c.max_batch * (size_t)l.nodes_per_utt * sizeof(TrieNode));
  l.state = off;
  if (c.max_chunk_frames > 0) off += up((size_t)c.max_batch * state_words(c.beam_width) * 4);
  l.beam_state = off;  // survivor lists (if any) + trie arenas + stream states
  l.stats = off; off += up((size_t)c.max_batch * kStatWords * sizeof(int32_t));
  l.flags = off; off += up(sizeof(int32_t));  // device-side error word of the prune kernel
  l.total = off;
  return l;
}

int cuda_fail(fltop_handle* h, cudaError_t e) {
  if (h) h->last_cuda = (int)e;
  cudaGetLastError();  // clear the sticky-free error state
  return FLTOP_ERR_CUDA;
}

struct DeviceGuard {
  int prev = -1;
  bool changed = false;
  cudaError_t enter(int dev) {
    cudaError_t e = cudaGetDevice(&prev);
    if (e != cudaSuccess) return e;
    if (prev != dev) {
      e = cudaSetDevice(dev);
      changed = (e == cudaSuccess);
    }
    return e;
  }
  ~DeviceGuard() {
    if (changed) cudaSetDevice(prev);
  }
};

int run_decode(fltop_handle* h, const void* d_logp, int64_t stride_b, int64_t stride_t,
               const int32_t* d_lengths, const uint8_t* d_flags, int32_t B, int32_t T,
               bool streaming, int32_t* d_tokens, int32_t* d_lens, float* d_scores,
               int32_t* d_nhyp, int32_t* d_status, cudaStream_t s, int32_t slot0 = 0,
               int32_t co_resident = 0) {
  // slot0: first of the handle's per-utterance scratch slots this launch uses (a batch that is
  // decoded group by group gives every group its own range of slots)
  DeviceGuard g;
  cudaError_t e = g.enter(h->cfg.device);
  if (e != cudaSuccess) return cuda_fail(h, e);
  h->prof_valid = false;
  if (B == 0) return FLTOP_OK;

  const bool fuse = h->fusion != 0 && T > 0 &&
                    decode_can_prune(h->cfg.vocab_size, h->cfg.emission_dtype, d_logp, stride_b, stride_t,
                                     h->cfg.top_n);
  if (!fuse && T > 0 && !h->counts) {
    // the first call that needs the separate prune kernel: its survivor lists are allocated now
    void* ptr = nullptr;
    e = cudaMalloc(&ptr, h->survivor_bytes);
    if (e != cudaSuccess) {
      cudaGetLastError();
      return e == cudaErrorMemoryAllocation ? FLTOP_ERR_OOM : cuda_fail(h, e);
    }
    h->survivor_extra = static_cast<unsigned char*>(ptr);
    h->counts = reinterpret_cast<int32_t*>(h->survivor_extra);
    h->entries = reinterpret_cast<Survivor*>(h->survivor_extra + h->counts_bytes);
    h->beam_state_bytes += h->survivor_bytes;
  }

  PruneParams pp = {};
  pp.error = h->prune_error;
  pp.staged = h->hook_prune_staged;
  pp.logp = d_logp; pp.dtype = h->cfg.emission_dtype;
  pp.stride_b = stride_b; pp.stride_t = stride_t; pp.lengths = d_lengths;
  pp.B = B; pp.T = T; pp.V = h->cfg.vocab_size; pp.log_r = h->log_r;
  pp.counts = h->counts ? h->counts + (int64_t)slot0 * T : nullptr;
  pp.entries = h->entries ? h->entries + (int64_t)slot0 * T * h->cfg.vocab_size : nullptr;

  DecodeParams dp = {};
  dp.lengths = d_lengths; dp.flags = d_flags; dp.B = B; dp.T = T; dp.V = h->cfg.vocab_size;
  dp.K = h->cfg.beam_width; dp.blank = h->cfg.blank_id; dp.L = h->cfg.max_out_len;
  dp.streaming = streaming ? 1 : 0; dp.emit_default = 1;
  dp.block_threads = h->block_threads; dp.warp_mode = h->warp_mode; dp.co_resident = co_resident; dp.pruning = h->cfg.threshold_r >= 5e-4f ? 1 : 0;  // weaker thresholds keep most tokens
  dp.top_n = h->cfg.top_n; dp.beam_threshold = h->cfg.beam_threshold;
  dp.merge_max = h->cfg.merge_max;
  dp.counts = pp.counts; dp.entries = pp.entries;
  dp.nodes = h->nodes + (int64_t)slot0 * h->nodes_per_utt;
  dp.logp = fuse ? d_logp : nullptr; dp.dtype = h->cfg.emission_dtype;
  dp.stride_b = stride_b; dp.stride_t = stride_t;
  dp.log_r = h->log_r;
  dp.nodes_per_utt = h->nodes_per_utt; dp.state = h->state;
  dp.out_tokens = d_tokens; dp.out_lens = d_lens; dp.out_scores = d_scores; dp.out_nhyp = d_nhyp;
  dp.out_status = d_status;
  dp.stats = h->stats + (int64_t)slot0 * kStatWords;
  dp.table_slots = h->hook_table_slots;
  dp.dbg_masks = h->hook_masks ? h->hook_masks + (int64_t)slot0 * T : nullptr;
  dp.dbg_clocks = slot0 == 0 ? h->hook_clocks : nullptr;
  dp.dbg_frame0 = h->hook_frame0; dp.dbg_frames = h->hook_frames;
  if (slot0 == 0) { h->last_B = B; h->last_T = T; h->last_stream = s; h->last_fused = fuse; }

  // (a batch decoded group by group on several streams is not timed kernel by kernel)
  const bool timed = h->profiling && co_resident == 0;
  if (timed) cudaEventRecord(h->ev[0], s);
  if (T > 0 && !fuse) {
    e = launch_prune(pp, s);
    if (e != cudaSuccess) return cuda_fail(h, e);
    ++h->launches;
    if (h->cfg.top_n > 0 && h->cfg.top_n < h->cfg.vocab_size) {
      e = launch_topn_cap(pp, h->cfg.top_n, s);
      if (e != cudaSuccess) return cuda_fail(h, e);
      ++h->launches;
    }
  }
  if (timed) cudaEventRecord(h->ev[1], s);
  if (decode_warp_eligible(dp)) e = launch_decode_warp(dp, s);
  else if (decode_rows_eligible(dp) && h->rows_mode != 0) e = launch_decode_rows(dp, s);
  else e = launch_decode(dp, s);
  if (e != cudaSuccess) return cuda_fail(h, e);
  ++h->launches;
  if (timed) {
    cudaEventRecord(h->ev[2], s);
    h->prof_valid = true;
  }
  return FLTOP_OK;
}

void host_io_release(HostIo& io) {
  for (int i = 0; i < kIoStreams; ++i) {
    if (io.stream[i]) cudaStreamDestroy(io.stream[i]);
    if (io.end[i]) cudaEventDestroy(io.end[i]);
  }
  for (int i = 0; i < kIoMaxGroups; ++i)
    if (io.done[i]) cudaEventDestroy(io.done[i]);
  if (io.begin) cudaEventDestroy(io.begin);
  if (io.dev) cudaFree(io.dev);
  if (io.pinned) cudaFreeHost(io.pinned);
  delete[] io.order;
  io = HostIo();
}

}  // namespace

extern "C" {

int fltop_enable_host_io(fltop_handle* h) {
  if (!h) return FLTOP_ERR_INVALID_ARG;
  if (h->cfg.max_chunk_frames > 0) return FLTOP_ERR_STATE;
  if (h->io.ready) return FLTOP_OK;
  DeviceGuard g;
  cudaError_t e = g.enter(h->cfg.device);
  if (e != cudaSuccess) return cuda_fail(h, e);
  HostIo& io = h->io;
  const size_t B = (size_t)h->cfg.max_batch, K = (size_t)h->cfg.beam_width;
  const size_t L = (size_t)h->cfg.max_out_len;
  const size_t n_logp = B * (size_t)h->cfg.max_frames * (size_t)h->cfg.vocab_size;
  size_t off = 0;
  const size_t o_logp = off; off += up(n_logp * emission_bytes(h->cfg.emission_dtype));
  const size_t o_len = off; off += up(B * 4);
  const size_t o_tok = off; off += up(B * K * L * 4);
  const size_t o_small = off; off += up(B * (2 * K + 2) * 4);
  void* ptr = nullptr;
  e = cudaMalloc(&ptr, off);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return e == cudaErrorMemoryAllocation ? FLTOP_ERR_OOM : cuda_fail(h, e);
  }
  io.dev = static_cast<unsigned char*>(ptr);
  io.d_logp = io.dev + o_logp;
  io.d_lengths = reinterpret_cast<int32_t*>(io.dev + o_len);
  io.d_tokens = reinterpret_cast<int32_t*>(io.dev + o_tok);
  io.d_small = reinterpret_cast<int32_t*>(io.dev + o_small);
  size_t poff = 0;
  const size_t q_len = poff; poff += up(B * 4);
  const size_t q_small = poff; poff += up(B * (2 * K + 2) * 4);
  e = cudaHostAlloc(&ptr, poff, cudaHostAllocDefault);
  if (e == cudaSuccess) {
    io.pinned = static_cast<unsigned char*>(ptr);
    io.p_lengths = reinterpret_cast<int32_t*>(io.pinned + q_len);
    io.p_small = reinterpret_cast<int32_t*>(io.pinned + q_small);
    io.order = new (std::nothrow) int32_t[B];
    if (!io.order) e = cudaErrorMemoryAllocation;
  }
  for (int i = 0; i < kIoStreams && e == cudaSuccess; ++i) {
    e = cudaStreamCreateWithFlags(&io.stream[i], cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&io.end[i], cudaEventDisableTiming);
  }
  for (int i = 0; i < kIoMaxGroups && e == cudaSuccess; ++i)
    e = cudaEventCreateWithFlags(&io.done[i], cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&io.begin, cudaEventDisableTiming);
  if (e != cudaSuccess) {
    host_io_release(io);
    return e == cudaErrorMemoryAllocation ? FLTOP_ERR_OOM : cuda_fail(h, e);
  }
  io.ready = true;
  return FLTOP_OK;
}

int fltop_decode_host(fltop_handle* h, const void* h_logp, int64_t stride_b, int64_t stride_t,
                      const int32_t* h_lengths, int32_t B, int32_t T, int32_t* h_tokens,
                      int32_t* h_lens, float* h_scores, int32_t* h_nhyp, int32_t* h_status,
                      void* cuda_stream) {
  if (!h) return FLTOP_ERR_INVALID_ARG;
  if (h->cfg.max_chunk_frames > 0 || !h->io.ready) return FLTOP_ERR_STATE;
  if (B < 0 || T < 0) return FLTOP_ERR_INVALID_ARG;
  if (B > h->cfg.max_batch || T > h->cfg.max_frames) return FLTOP_ERR_CAPACITY;
  if (B > 0 && (!h_lengths || !h_tokens || !h_lens || !h_scores || !h_nhyp))
    return FLTOP_ERR_INVALID_ARG;
  if (B > 0 && T > 0 && (!h_logp || stride_t < h->cfg.vocab_size || stride_b < 0))
    return FLTOP_ERR_INVALID_ARG;
  HostIo& io = h->io;
  io.h2d_bytes = io.d2h_bytes = 0;
  if (B == 0) return FLTOP_OK;
  DeviceGuard g;
  cudaError_t e = g.enter(h->cfg.device);
  if (e != cudaSuccess) return cuda_fail(h, e);
  cudaStream_t user = static_cast<cudaStream_t>(cuda_stream);
  const int64_t V = h->cfg.vocab_size, K = h->cfg.beam_width, L = h->cfg.max_out_len;

  // The longest utterances go first: the call lasts as long as the longest frame chain, so that
  // chain has to start as early as possible; everything else overlaps with it.
  auto usable = [&](int32_t u) -> int64_t {
    const int32_t len = h_lengths[u];
    return (len < 0 || len > T) ? 0 : len;  // the kernel flags such an utterance itself
  };
  for (int32_t i = 0; i < B; ++i) io.order[i] = i;
  std::stable_sort(io.order, io.order + B,
                   [&](int32_t a, int32_t b) { return usable(a) > usable(b); });
  for (int32_t i = 0; i < B; ++i) io.p_lengths[i] = h_lengths[io.order[i]];

  // Groups of utterances, in slot order.  The first group (the longest utterances) is a
  // quarter of the others: its copies are the head and the tail of the call that nothing
  // overlaps with.
  int32_t group = kIoGroupSize;
  if ((B + group - 1) / group + 1 > kIoMaxGroups)
    group = (B + kIoMaxGroups - 2) / (kIoMaxGroups - 1);
  const int32_t first = std::min(B, std::max(1, group / 4));
  const int32_t n_groups = 1 + (B - first + group - 1) / group;
  auto group_begin = [&](int32_t gi) -> int32_t {
    return gi == 0 ? 0 : std::min(B, first + (gi - 1) * group);
  };

  e = cudaEventRecord(io.begin, user);
  for (int i = 0; i < n_groups && e == cudaSuccess; ++i)
    e = cudaStreamWaitEvent(io.stream[i], io.begin, 0);
  if (e != cudaSuccess) return cuda_fail(h, e);

  int rc = FLTOP_OK;
  const int64_t row_pitch = (int64_t)T * V;  // device staging: [slot, T, V], this call's T
  const int64_t esize = (int64_t)emission_bytes(h->cfg.emission_dtype);
  const unsigned char* const h_bytes = static_cast<const unsigned char*>(h_logp);
  for (int32_t gi = 0; gi < n_groups && rc == FLTOP_OK; ++gi) {
    const int32_t s0 = group_begin(gi), n = group_begin(gi + 1) - s0;
    cudaStream_t st = io.stream[gi];
    e = cudaMemcpyAsync(io.d_lengths + s0, io.p_lengths + s0, (size_t)n * 4,
                        cudaMemcpyHostToDevice, st);
    io.h2d_bytes += (int64_t)n * 4;
    for (int32_t slot = s0; slot < s0 + n && e == cudaSuccess; ++slot) {
      const int32_t u = io.order[slot];
      const int64_t len = usable(u);
      if (len == 0) continue;
      unsigned char* dst = io.d_logp + (int64_t)slot * row_pitch * esize;
      const unsigned char* src = h_bytes + (int64_t)u * stride_b * esize;
      if (stride_t == V) {
        e = cudaMemcpyAsync(dst, src, (size_t)(len * V * esize), cudaMemcpyHostToDevice, st);
      } else {
        e = cudaMemcpy2DAsync(dst, (size_t)(V * esize), src, (size_t)(stride_t * esize),
                              (size_t)(V * esize), (size_t)len, cudaMemcpyHostToDevice, st);
      }
      io.h2d_bytes += len * V * esize;
    }
    if (e != cudaSuccess) { rc = cuda_fail(h, e); break; }
    int32_t* const small = io.d_small + (int64_t)s0 * (2 * K + 2);
    rc = run_decode(h, io.d_logp + (int64_t)s0 * row_pitch * esize, row_pitch, V, io.d_lengths + s0,
                    nullptr, n, T, false, io.d_tokens + (int64_t)s0 * K * L, small,
                    reinterpret_cast<float*>(small + (int64_t)n * K), small + (int64_t)2 * n * K,
                    small + (int64_t)2 * n * K + n, st, s0, B);
  }
  // The small outputs come home in the order the groups will finish, shortest first: copies
  // wait in the copy engine's queue in the order they were issued, and one that waits for a
  // long kernel would hold up those behind it.
  for (int32_t gi = n_groups - 1; gi >= 0 && rc == FLTOP_OK; --gi) {
    const int32_t s0 = group_begin(gi), n = group_begin(gi + 1) - s0;
    e = cudaMemcpyAsync(io.p_small + (int64_t)s0 * (2 * K + 2),
                        io.d_small + (int64_t)s0 * (2 * K + 2), (size_t)(n * (2 * K + 2)) * 4,
                        cudaMemcpyDeviceToHost, io.stream[gi]);
    if (e == cudaSuccess) e = cudaEventRecord(io.done[gi], io.stream[gi]);
    io.d2h_bytes += (int64_t)n * (2 * K + 2) * 4;
    if (e != cudaSuccess) rc = cuda_fail(h, e);
  }
  h->last_B = B; h->last_T = T; h->last_stream = user; h->prof_valid = false;

  // Results, shortest utterances (the last group) first: they are done long before the
  // longest.  Only the tokens that exist cross the bus: hypotheses x longest hypothesis.
  for (int32_t gi = n_groups - 1; gi >= 0 && rc == FLTOP_OK; --gi) {
    const int32_t s0 = group_begin(gi), n = group_begin(gi + 1) - s0;
    e = cudaEventSynchronize(io.done[gi]);
    const int32_t* const small = io.p_small + (int64_t)s0 * (2 * K + 2);
    const int32_t* const g_lens = small;
    const float* const g_scores = reinterpret_cast<const float*>(small + (int64_t)n * K);
    const int32_t* const g_nhyp = small + (int64_t)2 * n * K;
    const int32_t* const g_status = g_nhyp + n;
    for (int32_t slot = s0; slot < s0 + n && e == cudaSuccess; ++slot) {
      const int32_t u = io.order[slot], i = slot - s0;
      const int32_t nh = std::max(0, std::min<int32_t>(g_nhyp[i], (int32_t)K));
      h_nhyp[u] = g_nhyp[i];
      if (h_status) h_status[u] = g_status[i];
      int32_t longest = 0;
      for (int64_t k = 0; k < K; ++k) {
        const int32_t len = g_lens[(int64_t)i * K + k];
        h_lens[(int64_t)u * K + k] = len;
        h_scores[(int64_t)u * K + k] = g_scores[(int64_t)i * K + k];
        if (k < nh) longest = std::max(longest, len);
      }
      longest = (int32_t)std::min<int64_t>(longest, L);
      if (nh > 0 && longest > 0) {
        e = cudaMemcpy2DAsync(h_tokens + (int64_t)u * K * L, (size_t)L * 4,
                              io.d_tokens + (int64_t)slot * K * L, (size_t)L * 4,
                              (size_t)longest * 4, (size_t)nh, cudaMemcpyDeviceToHost,
                              io.stream[gi]);
        io.d2h_bytes += (int64_t)longest * nh * 4;
      }
    }
    if (e != cudaSuccess) rc = cuda_fail(h, e);
  }
  // the caller's stream resumes after everything; the host returns with the outputs in place
  for (int i = 0; i < n_groups; ++i) {
    e = cudaEventRecord(io.end[i], io.stream[i]);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(user, io.end[i], 0);
    if (e != cudaSuccess && rc == FLTOP_OK) rc = cuda_fail(h, e);
  }
  e = cudaStreamSynchronize(user);
  if (e != cudaSuccess && rc == FLTOP_OK) rc = cuda_fail(h, e);
  if (rc != FLTOP_OK)  // leave nothing of this call in flight
    for (int i = 0; i < n_groups; ++i) cudaStreamSynchronize(io.stream[i]);
  return rc;
}

int fltop_last_host_io_bytes(const fltop_handle* h, int64_t* out) {
  if (!h || !out) return FLTOP_ERR_INVALID_ARG;
  out[0] = h->io.h2d_bytes;
  out[1] = h->io.d2h_bytes;
  return FLTOP_OK;
}

size_t fltop_workspace_size(const fltop_config* cfg) {
  if (!config_ok(cfg)) return 0;
  return layout_of(*cfg).total;
}

int fltop_create(const fltop_config* cfg, fltop_handle** out) {
  if (!out) return FLTOP_ERR_INVALID_ARG;
  *out = nullptr;
  if (!config_ok(cfg)) return FLTOP_ERR_INVALID_ARG;
  const Layout l = layout_of(*cfg);
  if (cfg->workspace && cfg->workspace_bytes < l.total) return FLTOP_ERR_OOM;

  int n_dev = 0;
  cudaError_t e = cudaGetDeviceCount(&n_dev);
  if (e != cudaSuccess) { cudaGetLastError(); return FLTOP_ERR_CUDA; }
  if (cfg->device >= n_dev) return FLTOP_ERR_INVALID_ARG;
  DeviceGuard g;
  e = g.enter(cfg->device);
  if (e != cudaSuccess) { cudaGetLastError(); return FLTOP_ERR_CUDA; }

  fltop_handle* h = new (std::nothrow) fltop_handle();
  if (!h) return FLTOP_ERR_OOM;
  h->cfg = *cfg;
  h->log_r = cfg->threshold_r > 0.f ? (float)std::log((double)cfg->threshold_r)
                                    : -std::numeric_limits<float>::infinity();
  h->last_cuda = 0; h->launches = 0; h->profiling = false; h->prof_valid = false;
  h->block_threads = 0;
  h->fusion = 1;
  h->warp_mode = 1;
  h->rows_mode = 1;
  h->hook_masks = nullptr; h->hook_clocks = nullptr;
  h->hook_frame0 = h->hook_frames = h->hook_table_slots = h->hook_prune_staged = 0;
  h->ev[0] = h->ev[1] = h->ev[2] = nullptr;
  if (cfg->workspace) {
    h->ws = static_cast<unsigned char*>(cfg->workspace);
    h->owns_workspace = false;
  } else {
    void* ptr = nullptr;
    e = cudaMalloc(&ptr, l.total);
    if (e != cudaSuccess) {
      cudaGetLastError();
      delete h;
      return e == cudaErrorMemoryAllocation ? FLTOP_ERR_OOM : FLTOP_ERR_CUDA;
    }
    h->ws = static_cast<unsigned char*>(ptr);
    h->owns_workspace = true;
  }
  h->ws_bytes = l.total;
  h->survivor_extra = nullptr;
  h->survivor_bytes = l.survivor_bytes;
  h->counts_bytes = l.counts_bytes;
  h->counts = l.survivors_inside ? reinterpret_cast<int32_t*>(h->ws + l.survivors) : nullptr;
  h->entries = l.survivors_inside
                   ? reinterpret_cast<Survivor*>(h->ws + l.survivors + l.counts_bytes) : nullptr;
  h->nodes = reinterpret_cast<TrieNode*>(h->ws + l.nodes);
  h->state = cfg->max_chunk_frames > 0 ? reinterpret_cast<int32_t*>(h->ws + l.state) : nullptr;
  h->stats = reinterpret_cast<int32_t*>(h->ws + l.stats);
  h->prune_error = reinterpret_cast<int32_t*>(h->ws + l.flags);
  h->last_B = 0; h->last_T = 0; h->last_stream = nullptr; h->last_fused = false;
  h->frame_cap = l.frame_cap;
  h->nodes_per_utt = l.nodes_per_utt;
  h->beam_state_bytes = l.beam_state;
  e = decode_prepare(cfg->beam_width, cfg->vocab_size);
  if (e == cudaSuccess) e = cudaMemset(h->prune_error, 0, sizeof(int32_t));
  if (e == cudaSuccess && h->state) {
    // an un-reset stream holds an empty beam rather than garbage
    e = cudaMemset(h->state, 0, (size_t)cfg->max_batch * state_words(cfg->beam_width) * 4);
  }
  if (e != cudaSuccess) {
    cudaGetLastError();
    if (h->owns_workspace) cudaFree(h->ws);
    delete h;
    return FLTOP_ERR_CUDA;
  }
  *out = h;
  return FLTOP_OK;
}

int fltop_decode(fltop_handle* h, const void* d_logp, int64_t stride_b, int64_t stride_t,
                 const int32_t* d_lengths, int32_t B, int32_t T, int32_t* d_tokens,
                 int32_t* d_lens, float* d_scores, int32_t* d_nhyp, int32_t* d_status,
                 void* cuda_stream) {
  if (!h) return FLTOP_ERR_INVALID_ARG;
  if (h->cfg.max_chunk_frames > 0) return FLTOP_ERR_STATE;
  if (B < 0 || T < 0) return FLTOP_ERR_INVALID_ARG;
  if (B > h->cfg.max_batch || T > h->cfg.max_frames) return FLTOP_ERR_CAPACITY;
  if (B > 0 && (!d_lengths || !d_tokens || !d_lens || !d_scores || !d_nhyp))
    return FLTOP_ERR_INVALID_ARG;
  if (B > 0 && T > 0 && (!d_logp || stride_t < h->cfg.vocab_size || stride_b < 0))
    return FLTOP_ERR_INVALID_ARG;
  return run_decode(h, d_logp, stride_b, stride_t, d_lengths, nullptr, B, T, false, d_tokens,
                    d_lens, d_scores, d_nhyp, d_status, static_cast<cudaStream_t>(cuda_stream));
}

int fltop_stream_step(fltop_handle* h, const void* d_chunk, const int32_t* d_chunk_lens,
                      const uint8_t* d_flags, int32_t S, int32_t C, int32_t* d_tokens,
                      int32_t* d_lens, float* d_scores, int32_t* d_nhyp, int32_t* d_status,
                      void* cuda_stream) {
  if (!h) return FLTOP_ERR_INVALID_ARG;
  if (h->cfg.max_chunk_frames <= 0) return FLTOP_ERR_STATE;
  if (S < 0 || C < 0) return FLTOP_ERR_INVALID_ARG;
  if (S > h->cfg.max_batch || C > h->cfg.max_chunk_frames) return FLTOP_ERR_CAPACITY;
  if (S > 0 && !d_chunk_lens) return FLTOP_ERR_INVALID_ARG;
  if (S > 0 && C > 0 && !d_chunk) return FLTOP_ERR_INVALID_ARG;
  const int n_out = (d_tokens ? 1 : 0) + (d_lens ? 1 : 0) + (d_scores ? 1 : 0) + (d_nhyp ? 1 : 0);
  if (n_out != 0 && n_out != 4) return FLTOP_ERR_INVALID_ARG;
  const int64_t V = h->cfg.vocab_size;
  return run_decode(h, d_chunk, (int64_t)C * V, V, d_chunk_lens, d_flags, S, C, true, d_tokens,
                    d_lens, d_scores, d_nhyp, d_status, static_cast<cudaStream_t>(cuda_stream));
}

int fltop_prune(fltop_handle* h, const void* d_logp, int64_t stride_b, int64_t stride_t,
                const int32_t* d_lengths, int32_t B, int32_t T, int32_t* d_counts,
                void* d_entries, void* cuda_stream) {
  if (!h) return FLTOP_ERR_INVALID_ARG;
  if (B < 0 || T < 0) return FLTOP_ERR_INVALID_ARG;
  if (B == 0 || T == 0) return FLTOP_OK;
  if (!d_logp || !d_lengths || !d_counts || !d_entries) return FLTOP_ERR_INVALID_ARG;
  if (stride_t < h->cfg.vocab_size || stride_b < 0) return FLTOP_ERR_INVALID_ARG;
  DeviceGuard g;
  cudaError_t e = g.enter(h->cfg.device);
  if (e != cudaSuccess) return cuda_fail(h, e);
  PruneParams pp = {};
  pp.error = h->prune_error;
  pp.staged = h->hook_prune_staged;
  pp.logp = d_logp; pp.dtype = h->cfg.emission_dtype;
  pp.stride_b = stride_b; pp.stride_t = stride_t; pp.lengths = d_lengths;
  pp.B = B; pp.T = T; pp.V = h->cfg.vocab_size; pp.log_r = h->log_r;
  pp.counts = d_counts; pp.entries = static_cast<Survivor*>(d_entries);
  e = launch_prune(pp, static_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) return cuda_fail(h, e);
  ++h->launches;
  if (h->cfg.top_n > 0 && h->cfg.top_n < h->cfg.vocab_size) {
    e = launch_topn_cap(pp, h->cfg.top_n, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(h, e);
    ++h->launches;
  }
  return FLTOP_OK;
}

int fltop_destroy(fltop_handle* h) {
  if (!h) return FLTOP_ERR_INVALID_ARG;
  int rc = FLTOP_OK;
  DeviceGuard g;
  if (g.enter(h->cfg.device) != cudaSuccess) rc = FLTOP_ERR_CUDA;
  for (int i = 0; i < 3; ++i)
    if (h->ev[i]) cudaEventDestroy(h->ev[i]);
  host_io_release(h->io);
  if (h->survivor_extra && cudaFree(h->survivor_extra) != cudaSuccess) rc = FLTOP_ERR_CUDA;
  if (h->owns_workspace && h->ws && cudaFree(h->ws) != cudaSuccess) rc = FLTOP_ERR_CUDA;
  cudaGetLastError();
  delete h;
  return rc;
}

const char* fltop_status_string(int code) {
  switch (code) {
    case FLTOP_OK: return "ok";
    case FLTOP_ERR_INVALID_ARG: return "invalid argument";
    case FLTOP_ERR_CUDA: return "CUDA runtime error";
    case FLTOP_ERR_OOM: return "out of device memory or workspace too small";
    case FLTOP_ERR_CAPACITY: return "request exceeds the handle's capacity";
    case FLTOP_ERR_STATE: return "call not valid for this handle";
    default: return "unknown status";
  }
}

int fltop_last_cuda_error(const fltop_handle* h) { return h ? h->last_cuda : 0; }
size_t fltop_beam_state_bytes(const fltop_handle* h) { return h ? h->beam_state_bytes : 0; }
int64_t fltop_launch_count(const fltop_handle* h) { return h ? h->launches : 0; }

int fltop_last_call_stats(fltop_handle* h, int64_t* out) {
  if (!h || !out) return FLTOP_ERR_INVALID_ARG;
  for (int i = 0; i < 8; ++i) out[i] = 0;
  if (h->last_B == 0) return FLTOP_OK;
  DeviceGuard g;
  cudaError_t e = g.enter(h->cfg.device);
  if (e == cudaSuccess) e = cudaStreamSynchronize(h->last_stream);
  if (e != cudaSuccess) return cuda_fail(h, e);
  const size_t B = (size_t)h->last_B;
  // kernels that prune the frames themselves count the survivors; otherwise the prune kernel's
  // per-frame counts are summed
  const size_t n_frames = (h->last_fused || !h->counts) ? 0 : B * (size_t)h->last_T;
  int32_t* host = new (std::nothrow) int32_t[kStatWords * B + n_frames];
  if (!host) return FLTOP_ERR_OOM;
  e = cudaMemcpy(host, h->stats, kStatWords * B * sizeof(int32_t), cudaMemcpyDeviceToHost);
  if (e == cudaSuccess && n_frames)
    e = cudaMemcpy(host + kStatWords * B, h->counts, n_frames * sizeof(int32_t),
                   cudaMemcpyDeviceToHost);
  if (e == cudaSuccess) {
    for (size_t b = 0; b < B; ++b) {
      const int32_t* s = host + kStatWords * b;
      out[0] += s[0];
      out[2] += s[1];
      out[3] += s[2];
      out[4] = std::max<int64_t>(out[4], s[3]);
      out[5] += s[4];
      out[6] += s[5];
      if (h->last_fused) out[1] += s[6];
    }
    for (size_t i = 0; i < n_frames; ++i) out[1] += host[kStatWords * B + i];
  }
  delete[] host;
  if (e == cudaSuccess) {
    int32_t flag = 0;
    e = cudaMemcpy(&flag, h->prune_error, sizeof(flag), cudaMemcpyDeviceToHost);
    out[7] = flag;
  }
  if (e != cudaSuccess) return cuda_fail(h, e);
  return FLTOP_OK;
}

int fltop_set_test_hook(fltop_handle* h, int hook, void* d_buffer, int64_t a, int64_t b) {
  if (!h) return FLTOP_ERR_INVALID_ARG;
  switch (hook) {
    case FLTOP_HOOK_SURVIVOR_MASKS:
      h->hook_masks = static_cast<uint32_t*>(d_buffer);
      return FLTOP_OK;
    case FLTOP_HOOK_PHASE_CLOCKS:
      if (d_buffer && (a < 0 || b < 1 || b > (1 << 20))) return FLTOP_ERR_INVALID_ARG;
      h->hook_clocks = static_cast<long long*>(d_buffer);
      h->hook_frame0 = (int32_t)a;
      h->hook_frames = d_buffer ? (int32_t)b : 0;
      return FLTOP_OK;
    case FLTOP_HOOK_TABLE_SLOTS:
      if (a < 0 || a > (1 << 20) || (a & (a - 1)) != 0) return FLTOP_ERR_INVALID_ARG;
      h->hook_table_slots = (int32_t)a;
      return FLTOP_OK;
    case FLTOP_HOOK_ROW_KERNEL:
      if (a != 0 && a != 1) return FLTOP_ERR_INVALID_ARG;
      h->rows_mode = (int32_t)a;
      return FLTOP_OK;
    case FLTOP_HOOK_PRUNE_STAGING:
      if (a != 0 && a != 1) return FLTOP_ERR_INVALID_ARG;
      h->hook_prune_staged = (int32_t)a;
      return FLTOP_OK;
    default:
      return FLTOP_ERR_INVALID_ARG;
  }
}

int fltop_set_fusion(fltop_handle* h, int mode) {
  if (!h || (mode != 0 && mode != 1)) return FLTOP_ERR_INVALID_ARG;
  h->fusion = mode;
  return FLTOP_OK;
}

int fltop_set_warp_decode(fltop_handle* h, int mode) {
  if (!h || mode < 0 || mode > 2) return FLTOP_ERR_INVALID_ARG;
  h->warp_mode = mode;
  return FLTOP_OK;
}

int fltop_set_block_threads(fltop_handle* h, int32_t threads) {
  if (!h || threads < 0 || threads > 1024 || threads % 32 != 0) return FLTOP_ERR_INVALID_ARG;
  h->block_threads = threads;
  return FLTOP_OK;
}

int fltop_set_profiling(fltop_handle* h, int enable) {
  if (!h) return FLTOP_ERR_INVALID_ARG;
  if (enable && !h->ev[0]) {
    DeviceGuard g;
    cudaError_t e = g.enter(h->cfg.device);
    for (int i = 0; i < 3 && e == cudaSuccess; ++i) e = cudaEventCreate(&h->ev[i]);
    if (e != cudaSuccess) return cuda_fail(h, e);
  }
  h->profiling = enable != 0;
  h->prof_valid = false;
  return FLTOP_OK;
}

int fltop_last_kernel_ms(fltop_handle* h, float* out_ms) {
  if (!h || !out_ms) return FLTOP_ERR_INVALID_ARG;
  if (!h->profiling || !h->prof_valid) return FLTOP_ERR_STATE;
  cudaError_t e = cudaEventSynchronize(h->ev[2]);
  if (e == cudaSuccess) e = cudaEventElapsedTime(&out_ms[0], h->ev[0], h->ev[1]);
  if (e == cudaSuccess) e = cudaEventElapsedTime(&out_ms[1], h->ev[1], h->ev[2]);
  if (e != cudaSuccess) return cuda_fail(h, e);
  if (h->last_fused) out_ms[0] = 0.f;  // no prune kernel ran
  return FLTOP_OK;
}

}  // extern "C"
