// Internal declarations shared by the CUDA translation units of the library.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace fltop {

// One survivor of a frame: token id and its float32 log-probability.
struct __align__(8) Survivor {
  int32_t token;
  float logp;
};

// Prefix-trie node: a back-pointer record, written once when a prefix enters
// the beam and read only when hypotheses are written out.
struct __align__(8) TrieNode {
  int32_t parent;  // node id of the prefix without its last token, -1 for the root
  int32_t token;   // last token of the prefix, -1 for the root
};

// Per-stream state header kept in HBM between stream_step calls.
struct StateHeader {
  int32_t nbeam;      // live beam entries
  int32_t n_nodes;    // trie node ids handed out (node 0 = empty prefix)
  int32_t frames;     // frames consumed since the last reset
  int32_t status;     // sticky FLTOP_ST_* bits
  double offset;      // log-probability of the renormalisation point (see decode kernel)
  int32_t drift;      // float bits: how far blank-only frames have let the relative scores sink
                      // since the point was last moved (row kernel; 0 from the others)
  int32_t pad;
};
constexpr int kStateHeaderWords = sizeof(StateHeader) / 4;
// beam arrays stored after the header, each K words (fingerprints: 2K words each):
// node, last, len, pb, pnb, tot, fingerprint, parent fingerprint
constexpr int kStateWordsPerSlot = 10;
inline size_t state_words(int K) { return kStateHeaderWords + (size_t)kStateWordsPerSlot * K; }

// How the emissions are stored (FLTOP_EMISSION_* of the public header); always widened to
// float32 before anything is computed.
enum { kEmissionF32 = 0, kEmissionF16 = 1, kEmissionBF16 = 2 };
inline size_t emission_bytes(int dtype) { return dtype == kEmissionF32 ? 4 : 2; }

struct PruneParams {
  const void* logp;         // elements of `dtype`
  int32_t dtype;
  int64_t stride_b, stride_t;
  const int32_t* lengths;   // [B]
  int32_t B, T, V;
  float log_r;
  int32_t* counts;          // [B*T]
  Survivor* entries;        // [B*T*V]
  int32_t* error;           // one word, or-ed with 1 if a bounded wait on a bulk copy ran out; or null
  int32_t staged;           // 1: rows that qualify go through the shared-memory ring (bulk copies)
};

struct DecodeParams {
  const int32_t* lengths;   // [B] frames to consume in this call
  const uint8_t* flags;     // [B] streaming flags or null
  int32_t B, T, V, K, blank, L;
  int32_t streaming;        // 0: reset at entry, no state kept.  1: state loaded / stored
  int32_t emit_default;     // streaming with flags == null: emit results?
  int32_t block_threads;    // 0 = choose from K, V and whether pruning is on
  int32_t warp_mode;        // warp-per-utterance kernel: 0 never, 1 when it pays, 2 whenever it can
  int32_t co_resident;      // utterance blocks on the GPU at the same time as this launch's,
                            // its own included (0 = just its own B): launches of one batch
                            // split over several streams size their blocks for the whole batch
  int32_t first_wave;       // > 0: blocks take the utterances by length, the first `first_wave`
                            // blocks the longest (a batch of more utterances than SMs, at
                            // most 1024; see utterance_by_length)
  int32_t pruning;          // 1 when R is large enough that few tokens survive a frame
  int32_t top_n;            // survivors per frame are capped at this (0: no cap)
  float beam_threshold;     // kept prefixes score at least best - beam_threshold (<= 0: off)
  int32_t merge_max;        // 1: masses are combined by max instead of log-sum
  int32_t* counts;          // [B*T] survivors per frame (not touched by a kernel that prunes itself)
  const Survivor* entries;  // [B*T*V]
  // Non-null: the decode kernel prunes the rows itself (V <= 32) and `entries` is not read.
  const void* logp;         // elements of `dtype`
  int32_t dtype;
  int64_t stride_b, stride_t;
  float log_r;
  TrieNode* nodes;          // [B * nodes_per_utt]
  int64_t nodes_per_utt;
  int32_t* state;           // [B * state_words(K)] (streaming only)
  int32_t* out_tokens;      // [B,K,L] or null
  int32_t* out_lens;        // [B,K]
  float* out_scores;        // [B,K]
  int32_t* out_nhyp;        // [B]
  int32_t* out_status;      // [B] or null
  int32_t* stats;           // [B,kStatWords] (see below) or null
  int32_t table_slots;      // 0, or a power of two: the fingerprint table is cut down to this many
                            // slots (the test of the bounded probe walks makes it overflow)
  // instrumented instantiations (tests and profiling; null in every ordinary launch)
  uint32_t* dbg_masks;      // [B*T] survivor mask of every frame a decode kernel pruned itself
  long long* dbg_clocks;    // [dbg_frames][32 warps][8 phases] clock64 of block 0
  int32_t dbg_frame0, dbg_frames;
};
// per-utterance statistics of a call: frames, trie nodes created, sum of beam sizes, node ids
// used, fingerprint-tag clashes (probes that met another sequence with the same 20-bit tag),
// frames selected by the slow exact path, survivors over all frames (kernels that prune
// the frames themselves; the others leave the per-frame counts of the prune kernel)
constexpr int kStatWords = 8;

size_t decode_smem_bytes(int K, int V);
int decode_block_threads(int K, int V, bool pruning, int top_n, bool latency_bound);
cudaError_t launch_prune(const PruneParams& p, cudaStream_t s);
// keeps at most top_n survivors per frame (no-op for top_n <= 0 or >= V)
cudaError_t launch_topn_cap(const PruneParams& p, int top_n, cudaStream_t s);
cudaError_t launch_decode(const DecodeParams& p, cudaStream_t s);
// character vocabularies, beams up to 64, rows pruned inside (fltop_decode_rows.cu)
bool decode_rows_eligible(const DecodeParams& p);
cudaError_t launch_decode_rows(const DecodeParams& p, cudaStream_t s);
// narrow beams over narrow vocabularies: one warp per utterance (fltop_decode_warp.cu)
bool decode_warp_eligible(const DecodeParams& p);
cudaError_t launch_decode_warp(const DecodeParams& p, cudaStream_t s);
cudaError_t decode_prepare(int K, int V);  // one-time kernel attribute set-up
// the decode kernel can take these raw emission rows itself (strides in elements)
bool decode_can_prune(int V, int dtype, const void* logp, int64_t stride_b, int64_t stride_t,
                      int top_n);

}  // namespace fltop
