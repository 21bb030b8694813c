// fltop_decode_static: the batch decode for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they
// decode: a real-time audio thread that may not block on the driver's
// allocator, a plug-in that runs inside another framework's memory pool and
// was handed a fixed budget, code that runs after the process has already
// handed all device memory to its caching allocator.  For them the scratch
// that fltop_create would allocate (survivor lists and prefix-trie arena)
// lives in a fixed array in this file, compiled into the library image.
//
// The array's name is a host-side handle, not a device address, so the
// address is taken once per device with cudaGetSymbolAddress and only that
// pointer is handed to the kernels.
#include <cmath>
#include <limits>
#include <mutex>

#include "../../include/fltop.h"
#include "fltop_internal.h"

using namespace fltop;

namespace {

// Capacity of the fixed scratch (see fltop.h): frames, survivors and trie nodes.
constexpr int64_t kStaticMaxFrames = FLTOP_STATIC_MAX_FRAMES;
constexpr int64_t kStaticMaxVocab = FLTOP_STATIC_MAX_VOCAB;
constexpr int64_t kStaticMaxNodes = FLTOP_STATIC_MAX_NODES;
constexpr size_t kCountsBytes = (size_t)kStaticMaxFrames * sizeof(int32_t);
constexpr size_t kEntriesBytes = (size_t)kStaticMaxFrames * kStaticMaxVocab * sizeof(Survivor);
constexpr size_t kNodesBytes = (size_t)kStaticMaxNodes * sizeof(TrieNode);
constexpr size_t kScratchBytes = kCountsBytes + kEntriesBytes + kNodesBytes;
static_assert(kCountsBytes % 256 == 0 && kEntriesBytes % 256 == 0, "regions stay 256-byte aligned");

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_lock;
unsigned char* g_scratch_addr[kMaxDevices] = {nullptr};
// fixed layouts of the decode kernel whose launch attributes are set on a device (bits)
unsigned g_prepared[kMaxDevices] = {0u};

// Device address of the scratch on the current device, and the decode kernel ready to be
// launched for this beam width and vocabulary.  The first call per device (and per layout
// variant of the kernel) does the set-up: it may load the kernels and the array onto the
// device, so it belongs outside stream capture and outside real-time sections.
cudaError_t set_up(int device, int K, int V, unsigned char** out) {
  std::lock_guard<std::mutex> guard(g_setup_lock);
  if (!g_scratch_addr[device]) {
    void* ptr = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[device] = static_cast<unsigned char*>(ptr);
  }
  // Beams of at most 64 use one of two fixed layouts (vocabulary up to 32, or wider); their
  // attributes are set once.  Wider beams size their shared memory by the beam itself.
  const unsigned variant = K <= 64 ? (V <= 32 ? 1u : 2u) : 0u;
  if (variant == 0u || !(g_prepared[device] & variant)) {
    const cudaError_t e = decode_prepare(K, V);
    if (e != cudaSuccess) return e;
    g_prepared[device] |= variant;
  }
  *out = g_scratch_addr[device];
  return cudaSuccess;
}

}  // namespace

extern "C" int fltop_decode_static(int32_t vocab_size, int32_t blank_id, int32_t beam_width,
                                   float threshold_r, const float* d_logp, int64_t stride_b,
                                   int64_t stride_t, const int32_t* d_lengths, int32_t B, int32_t T,
                                   int32_t max_out_len, int32_t* d_tokens, int32_t* d_lens,
                                   float* d_scores, int32_t* d_nhyp, int32_t* d_status,
                                   void* cuda_stream) {
  if (vocab_size < 2 || blank_id < 0 || blank_id >= vocab_size || beam_width < 1 ||
      max_out_len < 1 || B < 0 || T < 0)
    return FLTOP_ERR_INVALID_ARG;
  if (!(threshold_r >= 0.f && threshold_r <= 1.f)) return FLTOP_ERR_INVALID_ARG;
  if (B == 0) return FLTOP_OK;
  if (!d_lengths || !d_tokens || !d_lens || !d_scores || !d_nhyp) return FLTOP_ERR_INVALID_ARG;
  if (T > 0 && (!d_logp || stride_t < vocab_size || stride_b < 0)) return FLTOP_ERR_INVALID_ARG;
  // the fixed scratch bounds the problem size
  const int64_t nodes_per_utt = (int64_t)((beam_width + 1) & ~1) * T + 2;
  if (vocab_size > kStaticMaxVocab || (int64_t)B * T > kStaticMaxFrames ||
      (int64_t)B * nodes_per_utt > kStaticMaxNodes)
    return FLTOP_ERR_CAPACITY;
  if (decode_smem_bytes(beam_width, vocab_size) > 227 * 1024) return FLTOP_ERR_CAPACITY;

  int device = 0;
  cudaError_t e = cudaGetDevice(&device);
  if (e != cudaSuccess || device >= kMaxDevices) { cudaGetLastError(); return FLTOP_ERR_CUDA; }
  unsigned char* scratch = nullptr;
  e = set_up(device, beam_width, vocab_size, &scratch);
  if (e != cudaSuccess) { cudaGetLastError(); return FLTOP_ERR_CUDA; }

  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  PruneParams pp = {};
  pp.logp = d_logp; pp.dtype = kEmissionF32; pp.stride_b = stride_b; pp.stride_t = stride_t; pp.lengths = d_lengths;
  pp.B = B; pp.T = T; pp.V = vocab_size;
  pp.log_r = threshold_r > 0.f ? (float)std::log((double)threshold_r)
                               : -std::numeric_limits<float>::infinity();
  pp.counts = reinterpret_cast<int32_t*>(scratch);
  pp.entries = reinterpret_cast<Survivor*>(scratch + kCountsBytes);

  DecodeParams dp = {};
  dp.lengths = d_lengths; dp.flags = nullptr; dp.B = B; dp.T = T; dp.V = vocab_size;
  dp.K = beam_width; dp.blank = blank_id; dp.L = max_out_len; dp.streaming = 0;
  dp.emit_default = 1; dp.block_threads = 0; dp.co_resident = 0; dp.warp_mode = 0; dp.pruning = threshold_r >= 5e-4f ? 1 : 0;
  dp.top_n = 0; dp.beam_threshold = 0.f; dp.merge_max = 0;
  dp.counts = pp.counts; dp.entries = pp.entries;
  dp.logp = nullptr; dp.dtype = kEmissionF32; dp.stride_b = 0; dp.stride_t = 0; dp.log_r = pp.log_r;
  dp.nodes = reinterpret_cast<TrieNode*>(scratch + kCountsBytes + kEntriesBytes);
  dp.nodes_per_utt = nodes_per_utt; dp.state = nullptr;
  dp.out_tokens = d_tokens; dp.out_lens = d_lens; dp.out_scores = d_scores; dp.out_nhyp = d_nhyp;
  dp.out_status = d_status; dp.stats = nullptr;

  // Nothing in the scratch has to start at zero: the prune kernel rewrites the count of
  // every frame of this call and the decode kernel re-creates each utterance's root node.
  if (T > 0) {
    e = launch_prune(pp, s);
    if (e != cudaSuccess) { cudaGetLastError(); return FLTOP_ERR_CUDA; }
  }
  e = launch_decode(dp, s);
  if (e != cudaSuccess) { cudaGetLastError(); return FLTOP_ERR_CUDA; }
  return FLTOP_OK;
}
