// Host side of the C ABI declared in include/fltop.h: argument validation,
// workspace carve-up and kernel launches on the caller's stream.
#include <cmath>
#include <limits>
#include <new>

#include "../../include/fltop.h"
#include "fltop_internal.h"

using namespace fltop;

struct fltop_handle {
  fltop_config cfg;
  float log_r;
  bool owns_workspace;
  unsigned char* ws;
  size_t ws_bytes;
  // regions of the workspace
  int32_t* counts;
  Survivor* entries;
  TrieNode* nodes;
  int32_t* state;
  int32_t* stats;
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
  bool profiling;
  bool prof_valid;
  cudaEvent_t ev[3];
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
  if (c->device < 0) return false;
  if ((int64_t)(c->beam_width + 1) * c->max_frames + 2 > (int64_t)std::numeric_limits<int32_t>::max())
    return false;
  if (decode_smem_bytes(c->beam_width, c->vocab_size) > kMaxSmem) return false;
  if (c->workspace && (reinterpret_cast<uintptr_t>(c->workspace) % kAlign) != 0) return false;
  return true;
}

struct Layout {
  size_t counts, entries, nodes, state, stats, total, beam_state;
  int64_t frame_cap, nodes_per_utt;
};

Layout layout_of(const fltop_config& c) {
  Layout l;
  l.frame_cap = c.max_chunk_frames > 0 ? c.max_chunk_frames : c.max_frames;
  // a frame takes an even-sized block of at most beam_width node ids; ids 0 and 1 are fixed
  l.nodes_per_utt = (int64_t)((c.beam_width + 1) & ~1) * c.max_frames + 2;
  const size_t frames = (size_t)c.max_batch * (size_t)l.frame_cap;
  size_t off = 0;
  l.counts = off; off += up(frames * sizeof(int32_t));
  l.entries = off; off += up(frames * (size_t)c.vocab_size * sizeof(Survivor));
  l.nodes = off; off += up((size_t)c.max_batch * (size_t)l.nodes_per_utt * sizeof(TrieNode));
  l.state = off;
  if (c.max_chunk_frames > 0) off += up((size_t)c.max_batch * state_words(c.beam_width) * 4);
  l.beam_state = off;  // survivor lists + trie arenas + stream states
  l.stats = off; off += up((size_t)c.max_batch * 4 * sizeof(int32_t));
  l.total = off;  // survivor lists + trie arenas + stream states
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

int run_decode(fltop_handle* h, const float* d_logp, int64_t stride_b, int64_t stride_t,
               const int32_t* d_lengths, const uint8_t* d_flags, int32_t B, int32_t T,
               bool streaming, int32_t* d_tokens, int32_t* d_lens, float* d_scores,
               int32_t* d_nhyp, int32_t* d_status, cudaStream_t s) {
  DeviceGuard g;
  cudaError_t e = g.enter(h->cfg.device);
  if (e != cudaSuccess) return cuda_fail(h, e);
  h->prof_valid = false;
  if (B == 0) return FLTOP_OK;

  PruneParams pp;
  pp.logp = d_logp; pp.stride_b = stride_b; pp.stride_t = stride_t; pp.lengths = d_lengths;
  pp.B = B; pp.T = T; pp.V = h->cfg.vocab_size; pp.log_r = h->log_r;
  pp.counts = h->counts; pp.entries = h->entries;

  DecodeParams dp;
  dp.lengths = d_lengths; dp.flags = d_flags; dp.B = B; dp.T = T; dp.V = h->cfg.vocab_size;
  dp.K = h->cfg.beam_width; dp.blank = h->cfg.blank_id; dp.L = h->cfg.max_out_len;
  dp.streaming = streaming ? 1 : 0; dp.emit_default = 1;
  dp.block_threads = h->block_threads; dp.pruning = h->cfg.threshold_r >= 5e-4f ? 1 : 0;  // weaker thresholds keep most tokens
  dp.top_n = h->cfg.top_n; dp.beam_threshold = h->cfg.beam_threshold;
  dp.counts = h->counts; dp.entries = h->entries; dp.nodes = h->nodes;
  const bool fuse = h->fusion != 0 && T > 0 && decode_can_prune(h->cfg.vocab_size);
  dp.logp = fuse ? d_logp : nullptr; dp.stride_b = stride_b; dp.stride_t = stride_t;
  dp.log_r = h->log_r;
  dp.nodes_per_utt = h->nodes_per_utt; dp.state = h->state;
  dp.out_tokens = d_tokens; dp.out_lens = d_lens; dp.out_scores = d_scores; dp.out_nhyp = d_nhyp;
  dp.out_status = d_status;
  dp.stats = h->stats;
  h->last_B = B; h->last_T = T; h->last_stream = s; h->last_fused = fuse;

  if (h->profiling) cudaEventRecord(h->ev[0], s);
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
  if (h->profiling) cudaEventRecord(h->ev[1], s);
  e = launch_decode(dp, s);
  if (e != cudaSuccess) return cuda_fail(h, e);
  ++h->launches;
  if (h->profiling) {
    cudaEventRecord(h->ev[2], s);
    h->prof_valid = true;
  }
  return FLTOP_OK;
}

}  // namespace

extern "C" {

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
  h->counts = reinterpret_cast<int32_t*>(h->ws + l.counts);
  h->entries = reinterpret_cast<Survivor*>(h->ws + l.entries);
  h->nodes = reinterpret_cast<TrieNode*>(h->ws + l.nodes);
  h->state = cfg->max_chunk_frames > 0 ? reinterpret_cast<int32_t*>(h->ws + l.state) : nullptr;
  h->stats = reinterpret_cast<int32_t*>(h->ws + l.stats);
  h->last_B = 0; h->last_T = 0; h->last_stream = nullptr; h->last_fused = false;
  h->frame_cap = l.frame_cap;
  h->nodes_per_utt = l.nodes_per_utt;
  h->beam_state_bytes = l.beam_state;
  e = decode_prepare(cfg->beam_width, cfg->vocab_size);
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

int fltop_decode(fltop_handle* h, const float* d_logp, int64_t stride_b, int64_t stride_t,
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

int fltop_stream_step(fltop_handle* h, const float* d_chunk, const int32_t* d_chunk_lens,
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

int fltop_prune(fltop_handle* h, const float* d_logp, int64_t stride_b, int64_t stride_t,
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
  PruneParams pp;
  pp.logp = d_logp; pp.stride_b = stride_b; pp.stride_t = stride_t; pp.lengths = d_lengths;
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
  out[0] = out[1] = out[2] = out[3] = 0;
  if (h->last_B == 0) return FLTOP_OK;
  DeviceGuard g;
  cudaError_t e = g.enter(h->cfg.device);
  if (e == cudaSuccess) e = cudaStreamSynchronize(h->last_stream);
  if (e != cudaSuccess) return cuda_fail(h, e);
  const size_t B = (size_t)h->last_B, n_frames = B * (size_t)h->last_T;
  int32_t* host = new (std::nothrow) int32_t[4 * B + n_frames];
  if (!host) return FLTOP_ERR_OOM;
  e = cudaMemcpy(host, h->stats, 4 * B * sizeof(int32_t), cudaMemcpyDeviceToHost);
  if (e == cudaSuccess && n_frames)
    e = cudaMemcpy(host + 4 * B, h->counts, n_frames * sizeof(int32_t), cudaMemcpyDeviceToHost);
  if (e == cudaSuccess) {
    for (size_t b = 0; b < B; ++b) {
      out[0] += host[4 * b];
      out[2] += host[4 * b + 1];
      out[3] += host[4 * b + 2];
    }
    for (size_t i = 0; i < n_frames; ++i) out[1] += host[4 * B + i];
  }
  delete[] host;
  if (e != cudaSuccess) return cuda_fail(h, e);
  return FLTOP_OK;
}

int fltop_set_fusion(fltop_handle* h, int mode) {
  if (!h || (mode != 0 && mode != 1)) return FLTOP_ERR_INVALID_ARG;
  h->fusion = mode;
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
