/*
 * fltop.h - C ABI of the frame-pruned CTC prefix beam search library (sm_100a).
 *
 * The library decodes frame-level log-probability emissions with the
 * procedure of the FLToP CTC paper (Algorithm 1): the beam starts with the
 * empty prefix; at every frame only tokens whose probability is at least R
 * times the frame's top probability extend the beam (the conditional break of
 * Algorithm 1, Section 3); candidates naming the same prefix are combined and
 * the best beam_size are kept (SelectTopK); after the last frame the
 * hypotheses are returned best first (GetHighestScorePrefix, widened to the
 * whole beam).  The CTC collapsing rule is the standard one of the "standard
 * BeamSearchCTC decoders" the paper modifies (Section 3): each prefix carries
 * the log-mass of alignments ending in blank and ending in its last token.
 * The top-N stage (N) and beam_threshold of Algorithm 1 are optional config
 * fields; its language model is not implemented.
 *
 * Conventions
 *   - every `d_*` pointer is DEVICE memory owned by the caller (`h_*`: HOST
 *     memory, fltop_decode_host only); the library never frees or keeps it
 *     beyond the call's work on `cuda_stream`.
 *   - calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*;
 *     NULL = the legacy default stream) and return without synchronising;
 *     outputs are valid once the caller has synchronised the stream.
 *   - the return value reports what the host can detect (bad arguments,
 *     capacity of the handle, CUDA launch errors).  Conditions only the
 *     device sees are reported per utterance in `d_status`.
 *   - no call prints, throws or aborts.  A handle must not be used from two
 *     threads at once; distinct handles are independent.
 */
#ifndef FLTOP_H_
#define FLTOP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fltop_handle fltop_handle; /* opaque, owned by the library */

enum {
  FLTOP_OK = 0,
  FLTOP_ERR_INVALID_ARG = 1, /* null pointer, value out of range, reserved field set */
  FLTOP_ERR_CUDA = 2,        /* a CUDA runtime call failed (see fltop_last_cuda_error) */
  FLTOP_ERR_OOM = 3,         /* workspace allocation failed or caller workspace too small */
  FLTOP_ERR_CAPACITY = 4,    /* B, T, S or C above what the handle was created for; per
                                utterance: trie arena full or output length above max_out_len */
  FLTOP_ERR_STATE = 5        /* call not valid for this handle (decode on a streaming
                                handle or the reverse) */
};

/* How the emissions are stored (fltop_config.emission_dtype).  Half-precision values are
 * widened to float32 (exactly) as they are loaded; everything else, the pruning comparison
 * included, is the float32 arithmetic described below.  Every `logp` / `chunk` pointer of
 * this header points to elements of the handle's emission_dtype; strides count elements. */
enum {
  FLTOP_EMISSION_F32 = 0,
  FLTOP_EMISSION_F16 = 1,    /* IEEE binary16 */
  FLTOP_EMISSION_BF16 = 2    /* bfloat16 */
};

/* Per-utterance device status bits written to d_status (0 = fine). */
enum {
  FLTOP_ST_BAD_LENGTH = 1,   /* length < 0 or > T: utterance skipped, nhyp = 0 */
  FLTOP_ST_ARENA_FULL = 2,   /* prefix trie arena exhausted: results of this utterance invalid */
  FLTOP_ST_TRUNCATED = 4,    /* a hypothesis is longer than max_out_len: tokens cut, lens true */
  FLTOP_ST_EMPTY_BEAM = 8,   /* every candidate had probability 0 (all -inf rows) */
  FLTOP_ST_INTERNAL = 16     /* a bounded device loop gave up; results invalid */
};

typedef struct {
  int32_t vocab_size;     /* V, 2 <= V <= 8192; V and K together must fit one SM's shared
                             memory (about 48 V + 130 K bytes <= 227 KB, plus 16 bytes a token
                             for 32 < V <= 1024, whose rows the decode block keeps four frames
                             of: V = 4096 with small beams, K = 1500 at V = 32), else
                             fltop_create refuses */
  int32_t blank_id;       /* 0 <= blank_id < V */
  int32_t beam_width;     /* K = beam_size of Algorithm 1, 1 <= K <= 2048 */
  float threshold_r;      /* R of Algorithm 1 in the probability domain, 0 <= R <= 1;
                             0 disables pruning.  A token survives a frame iff
                             logp >= logp_max + (float)log((double)R), float32 compare */
  int32_t max_batch;      /* capacity: utterances per fltop_decode call / concurrent streams */
  int32_t max_frames;     /* capacity: frames per utterance (decode) or per stream between
                             two resets (stream_step) */
  int32_t max_chunk_frames; /* 0: the handle serves fltop_decode.  > 0: the handle serves
                             fltop_stream_step with chunks of at most this many frames */
  int32_t max_out_len;    /* L of the token output, 1 <= L */
  int32_t top_n;          /* N of Algorithm 1 (PartialSortDesc): a frame keeps at most its
                             top_n most probable tokens, before R is applied; at a tie for
                             the last place the lower token id stays.  0 = no cap */
  float beam_threshold;   /* beam_threshold of Algorithm 1 (SelectTopK): of the beam_width
                             best prefixes of a frame, those scoring below best -
                             beam_threshold are dropped, so a beam can hold fewer than
                             beam_width prefixes.  <= 0 = no such cut */
  int32_t merge_max;      /* 0: candidates naming the same prefix, and a prefix' blank and
                             non-blank mass, are combined by log-sum (a prefix scores as the
                             sum over its alignments).  1: by max, Algorithm 1's literal
                             score' = score + logit: a prefix scores as its best alignment */
  int32_t emission_dtype; /* FLTOP_EMISSION_*: element type of the emissions */
  int32_t max_trie_nodes; /* capacity of ONE utterance's (stream's) prefix trie, in 8-byte nodes.
                             A node is created when a prefix enters the beam that was not in it
                             the frame before: at most beam_width per frame.  0 = that worst
                             case, beam_width x max_frames, which can never run out.  Peaked
                             emissions need far less (the character workload of the benchmark:
                             0.36 x beam_width per frame); a handle created with a smaller
                             capacity holds less memory, and an utterance that does run out is
                             reported with FLTOP_ST_ARENA_FULL, never written past the end */
  int32_t device;         /* CUDA device ordinal */
  void* workspace;        /* optional DEVICE memory, 256-byte aligned, for all of the
                             handle's scratch; NULL = the library allocates it */
  size_t workspace_bytes; /* size of `workspace`; ignored when workspace is NULL */
} fltop_config;

/* Bytes of device scratch a handle with this config needs (0 on invalid config). */
size_t fltop_workspace_size(const fltop_config* cfg);

/* Algorithm 1, procedure header: fixes beam_size, R and the shapes.  Validates cfg,
 * sizes and allocates (or adopts) the workspace.  On success *out is a new handle. */
int fltop_create(const fltop_config* cfg, fltop_handle** out);

/* Algorithm 1 for a whole batch.  Each of the B utterances is decoded independently.
 *   d_logp      [B,T,V] log-probabilities (emission_dtype); element strides stride_b, stride_t,
 *               the V entries of a frame contiguous.  Rows that start on a multiple of four
 *               elements' bytes, with V % 4 == 0, take the fast path.
 *               Frames t >= d_lengths[b] are never read.
 *   d_lengths   [B] int32 frame counts.
 *   d_tokens    [B,K,L] int32: hypothesis k of utterance b, L = max_out_len; entries past
 *               the hypothesis' length are left untouched.  Inside the search a prefix is
 *               identified by a 64-bit fingerprint of its token sequence: two different
 *               prefixes that are in the beam of the same frame and share all 64 bits would be
 *               taken for one (chance about 2^-64 per pair and frame; not detected).
 *   d_lens      [B,K] int32 true lengths (0 for unused slots k >= nhyp).
 *   d_scores    [B,K] float32 log-probability of each hypothesis (log-sum of its blank and
 *               non-blank mass at the last frame, the larger of the two with merge_max; -inf
 *               for unused slots); best first.  Hypotheses whose scores tie exactly come in
 *               no particular order.
 *   d_nhyp      [B] int32 number of hypotheses (<= K; 1 with the empty sequence and score 0
 *               when the length is 0).
 *   d_status    [B] int32 FLTOP_ST_* bits, may be NULL. */
int fltop_decode(fltop_handle* h, const void* d_logp, int64_t stride_b, int64_t stride_t,
                 const int32_t* d_lengths, int32_t B, int32_t T, int32_t* d_tokens,
                 int32_t* d_lens, float* d_scores, int32_t* d_nhyp, int32_t* d_status,
                 void* cuda_stream);

/* fltop_decode for callers whose emissions and results live in HOST memory (Algorithm 1 is
 * stated on host arrays; this is the same procedure with the transfers done by the library).
 * fltop_enable_host_io allocates, once, what that takes: device copies of the inputs and
 * outputs ([max_batch, max_frames, V] emissions + [max_batch, K, L] int32 + small arrays), a few
 * KB of pinned host memory, sixteen streams.  FLTOP_ERR_STATE on a streaming handle,
 * FLTOP_ERR_OOM / FLTOP_ERR_CUDA if an allocation fails (the handle stays usable for the
 * device-pointer calls); calling it again is a no-op. */
int fltop_enable_host_io(fltop_handle* h);

/* Arguments as in fltop_decode, but every h_* pointer is HOST memory (pinned memory lets the
 * copies run asynchronously; pageable memory works, slower).  The batch is cut into groups of
 * utterances, longest first; each group's frames are copied (only the h_lengths[b] valid frames
 * of an utterance), decoded and read back on streams of the handle, so that all transfers but
 * the first group's overlap with decoding.  Only existing tokens are copied back:
 * h_tokens[b,k,0:len] for k < nhyp is written, everything else in h_tokens is left untouched;
 * h_lens, h_scores, h_nhyp and (if not NULL) h_status are written in full.
 * The work is ordered after what `cuda_stream` held at the call and `cuda_stream` waits for
 * it; unlike the device-pointer calls this one RETURNS ONLY WHEN THE OUTPUTS ARE IN HOST
 * MEMORY.  Results are those of fltop_decode: the same scores bit for bit, the same hypotheses
 * up to the order of exactly tied ones.  (Up to 16 of the handle's streams
 * are busy at once; a process that leaves CUDA_DEVICE_MAX_CONNECTIONS at its default of 8 lets
 * them share hardware queues, which costs a few per cent.)  FLTOP_ERR_STATE unless
 * fltop_enable_host_io succeeded on this handle. */
int fltop_decode_host(fltop_handle* h, const void* h_logp, int64_t stride_b, int64_t stride_t,
                      const int32_t* h_lengths, int32_t B, int32_t T, int32_t* h_tokens,
                      int32_t* h_lens, float* h_scores, int32_t* h_nhyp, int32_t* h_status,
                      void* cuda_stream);
/* Bytes the most recent fltop_decode_host moved: out[0] host to device, out[1] device to host. */
int fltop_last_host_io_bytes(const fltop_handle* h, int64_t* out);

/* Algorithm 1 consumed chunk by chunk: the frame loop of S concurrent streams advances by
 * up to C frames; the beam of every stream is kept in the handle between calls.
 *   d_chunk      [S,C,V] emission_dtype, contiguous.
 *   d_chunk_lens [S] int32 valid frames of each stream in this chunk (0 = idle).
 *   d_flags      [S] uint8, may be NULL: bit0 = reset the stream to the empty prefix before
 *                consuming the chunk; bit1 = write this stream's current hypotheses.
 *                NULL means "no reset, write hypotheses if output pointers are given".
 *                A stream must be reset before its first chunk.
 *   outputs as in fltop_decode with B = S; all four may be NULL together (no readback). */
int fltop_stream_step(fltop_handle* h, const void* d_chunk, const int32_t* d_chunk_lens,
                      const uint8_t* d_flags, int32_t S, int32_t C, int32_t* d_tokens,
                      int32_t* d_lens, float* d_scores, int32_t* d_nhyp, int32_t* d_status,
                      void* cuda_stream);

/* Releases the handle and the workspace if the library allocated it. */
int fltop_destroy(fltop_handle* h);

/* The frame-level pruning step alone (Algorithm 1, conditional break), exactly as the two
 * calls above run it: for every frame the survivors in ascending token order.
 *   d_counts  [B,T] int32 survivors per frame (0 for frames past the length).
 *   d_entries [B,T,V] pairs {int32 token, float32 logp}; the first d_counts[b,t] pairs of
 *             frame (b,t) are valid. */
int fltop_prune(fltop_handle* h, const void* d_logp, int64_t stride_b, int64_t stride_t,
                const int32_t* d_lengths, int32_t B, int32_t T, int32_t* d_counts,
                void* d_entries, void* cuda_stream);

/* Batch decode without any allocation.  The paper has no counterpart to this call: it exists
 * for callers that cannot call cudaMalloc where they decode - a real-time audio thread that
 * must not block in the driver's allocator, a plug-in living inside another framework's
 * memory pool with a fixed budget, a process that has already given all device memory to a
 * caching allocator.  It computes exactly what fltop_create + fltop_decode + fltop_destroy
 * compute, but its scratch (survivor lists, prefix-trie arena) is a fixed array inside the
 * library image, FLTOP_STATIC_SCRATCH_BYTES per GPU that loads the library, held until the
 * process exits.  Consequently:
 *   - the problem must fit: vocab_size <= FLTOP_STATIC_MAX_VOCAB, B*T <=
 *     FLTOP_STATIC_MAX_FRAMES, B*(K2*T + 2) <= FLTOP_STATIC_MAX_NODES with K2 = beam_width
 *     rounded up to an even number; anything
 *     larger returns FLTOP_ERR_CAPACITY and launches nothing;
 *   - it runs on the CURRENT device.  The first call on each device looks up the array's
 *     device address (cudaGetSymbolAddress) and sets the decode kernel's launch attributes
 *     before launching (the latter again for a shape that needs another layout of the
 *     kernel); the driver may load the kernels and the array onto the device at that point.
 *     Make that first call - a warm-up - outside any stream capture and outside any
 *     real-time section;
 *   - all calls share the one array.  It needs no clearing between calls (every word a
 *     call reads it has written first), but two calls whose kernels overlap on the GPU -
 *     different streams, or different host threads - race on it.  Serialise them.
 *   - it calls no cudaMalloc / cudaFree and no allocating library routine; inputs and
 *     outputs are the caller's device buffers, with the meaning they have in fltop_decode
 *     (d_tokens is [B, beam_width, max_out_len]). */
#define FLTOP_STATIC_MAX_VOCAB 64
#define FLTOP_STATIC_MAX_FRAMES 4096
#define FLTOP_STATIC_MAX_NODES 131072
#define FLTOP_STATIC_SCRATCH_BYTES \
  (FLTOP_STATIC_MAX_FRAMES * 4 + FLTOP_STATIC_MAX_FRAMES * FLTOP_STATIC_MAX_VOCAB * 8 + \
   FLTOP_STATIC_MAX_NODES * 8)
int fltop_decode_static(int32_t vocab_size, int32_t blank_id, int32_t beam_width,
                        float threshold_r, const float* d_logp, int64_t stride_b,
                        int64_t stride_t, const int32_t* d_lengths, int32_t B, int32_t T,
                        int32_t max_out_len, int32_t* d_tokens, int32_t* d_lens, float* d_scores,
                        int32_t* d_nhyp, int32_t* d_status, void* cuda_stream);

/* Optional helpers. */
const char* fltop_status_string(int code);
/* Last cudaError_t seen by this handle (0 if none). */
int fltop_last_cuda_error(const fltop_handle* h);
/* Bytes of beam state the handle holds now: prefix trie arenas, stream states and - once a
 * call has needed them - the survivor lists of the separate prune kernel (vocabularies above
 * 1024 tokens get them at fltop_create; narrower ones only if a call cannot prune inside the
 * decode kernel, see fltop_set_fusion, and then by a device allocation of the library's own
 * even when the handle lives in a caller's workspace). */
size_t fltop_beam_state_bytes(const fltop_handle* h);
/* Kernels launched by this handle since creation. */
int64_t fltop_launch_count(const fltop_handle* h);
/* Totals of the most recent decode / stream_step call (synchronises its stream), eight values:
 * out[0] frames decoded, out[1] survivors over those frames, out[2] prefix-trie nodes
 * created, out[3] beam entries summed over frames (mean live hypotheses = out[3]/out[0]),
 * out[4] the largest number of trie node ids any one utterance has used so far, out[5] probes
 * of the fingerprint table that met a different prefix with the same 20-bit tag (each was
 * told apart by the full 64 bits), out[6] frames whose selection took the slow exact path,
 * out[7] non-zero if, since the handle was created, a bounded wait of the prune kernel on one of
 * its asynchronous row copies ran out (it does not spin forever; the rows left get no
 * survivors and the results of that call are invalid). */
int fltop_last_call_stats(fltop_handle* h, int64_t* out);
/* With profiling enabled every call brackets its kernels with CUDA events on the caller's
 * stream.  fltop_last_kernel_ms synchronises on those events and returns the device time
 * of the most recent call's {prune, decode} kernels in out_ms[0..1] (milliseconds); the
 * first is 0 when the decode kernel pruned the frames itself (see fltop_set_fusion). */
int fltop_set_profiling(fltop_handle* h, int enable);
/* Threads per utterance block of the decode kernel (a multiple of 32, at most 1024; 0 = let
 * the library choose from K, V and R).  A tuning knob: results do not depend on it. */
int fltop_set_block_threads(fltop_handle* h, int32_t threads);
/* Where the frames are pruned (Algorithm 1, the top-N stage and the conditional break).
 * mode 1 (the default): inside the decode kernel whenever it can - each utterance block (or
 * warp) fetches its own emission rows and no survivor list goes through device memory.  It
 * can for vocab_size <= 32 with any element type, and for vocab_size <= 1024 with float32
 * emissions whose rows start on 16-byte boundaries (vocab_size and both strides multiples of
 * four, d_logp 16-byte aligned) and no top_n cap.  Everything else takes the separate prune
 * kernel, which writes [B,T,V] survivor pairs that the decode kernel reads back.  mode 0:
 * always the separate kernel.  The survivors are the same bit for bit either way, the
 * hypotheses the same up to the order of exactly tied ones.  FLTOP_ERR_INVALID_ARG for a null handle or another mode. */
int fltop_set_fusion(fltop_handle* h, int mode);
/* Which decode kernel serves narrow problems (beam_width <= 32, vocab_size <= 32, pruning
 * inside the kernel, no beam_threshold, no merge_max, no block size set).  The library has two
 * kinds: one thread block per utterance, and one warp per utterance with several utterances to a block.
 * A warp alone is slower on its utterance but an SM runs many more of them side by side.
 * mode 1 (the default): the warp kernel when a call brings at least eight utterances or streams
 * per SM; mode 0: never; mode 2: whenever the problem is narrow enough.  Results are the same up
 * to the order of exactly tied hypotheses.  FLTOP_ERR_INVALID_ARG for another mode. */
int fltop_set_warp_decode(fltop_handle* h, int mode);
int fltop_last_kernel_ms(fltop_handle* h, float* out_ms);

/* Instrumented launches, for tests and profiling; everything is off on a new handle and no
 * ordinary launch pays for it.  The paper has no counterpart.
 *   FLTOP_HOOK_SURVIVOR_MASKS  d_buffer: DEVICE uint32 [B*T] of the next calls (NULL = off).
 *       A decode kernel that prunes the frames of a vocabulary of at most 32 tokens itself
 *       writes the survivor
 *       set of frame (b,t) - bit c set iff token c survives Algorithm 1's top-N stage and
 *       conditional break - to d_buffer[b*T + t]; frames past the length are left untouched.
 *   FLTOP_HOOK_PHASE_CLOCKS    d_buffer: DEVICE int64 [b][32][8] (NULL = off): for frames
 *       a <= t < a + b of utterance 0 the row kernel records the SM clock of every warp at its
 *       eight phase boundaries (frame start, end of evaluation, after the first barrier, after
 *       the histogram scan, end of placement, after the list barrier, before and after the
 *       last barrier).  The general block kernel (without beam_threshold / merge_max) records
 *       its own eight marks for the utterance of block 0: frame start, candidates evaluated,
 *       past the first barrier, cut known, candidates settled, at the second barrier (large
 *       blocks), next beam written, past the last barrier.
 *   FLTOP_HOOK_TABLE_SLOTS     a: 0 (off) or a power of two: the shared-memory table of prefix
 *       fingerprints is cut down to that many slots.  With fewer slots than beam entries its
 *       bounded probe walks run out, which the kernels report as FLTOP_ST_INTERNAL.
 *   FLTOP_HOOK_ROW_KERNEL      a: 1 (default) vocabularies of at most 32 tokens with beams of at
 *       most 128 take the row kernel; 0: they take the general block kernel.
 *   FLTOP_HOOK_PRUNE_STAGING   a: 1: the separate prune kernel stages rows of 1 to 4 KB through
 *       shared memory with asynchronous bulk copies instead of holding them in registers (same
 *       results; measured slower, kept for measurements); 0 (default): registers.
 * FLTOP_ERR_INVALID_ARG for a null handle, an unknown hook or a value out of range. */
enum {
  FLTOP_HOOK_SURVIVOR_MASKS = 1,
  FLTOP_HOOK_PHASE_CLOCKS = 2,
  FLTOP_HOOK_TABLE_SLOTS = 3,
  FLTOP_HOOK_ROW_KERNEL = 4,
  FLTOP_HOOK_PRUNE_STAGING = 5
};
int fltop_set_test_hook(fltop_handle* h, int hook, void* d_buffer, int64_t a, int64_t b);

#ifdef __cplusplus
}
#endif
#endif /* FLTOP_H_ */
