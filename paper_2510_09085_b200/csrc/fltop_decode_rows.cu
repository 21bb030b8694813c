// CTC prefix beam search over pruned frames for character vocabularies (at most 32 tokens)
// and beams of at most 128 prefixes: the shape the paper itself decodes (Section 4: 32 tokens).
// Algorithm 1 with the standard CTC collapsing rule, one thread block per utterance, frames
// walked serially, the beam in shared memory.
//
// A frame is a chain of dependent steps, so the design goal is the shortest chain, not
// bandwidth.  What differs from the general block kernel (fltop_decode.cu):
//
//   * One chore warp prepares frames ahead of their use.  A vocabulary of at most 32 tokens is
//     one token per lane: the row maximum is one warp reduction, the relative threshold
//     (Algorithm 1's conditional break) one float32 add and compare, the survivors one ballot.
//     What the other warps need of a frame (log-probability by token, the surviving non-blank
//     tokens in a row, which warp walks which of them) waits for them in a ring of four
//     frames; the same warp alone scans the score histogram and publishes the cut.
//   * A frame in which only blank survives changes no prefix: the beam is updated in place,
//     and the renormalisation that was skipped is carried as a drift term.
//   * Extension candidates are laid out as rows of "one surviving token x 32 beam entries": an
//     extension lane owns one beam entry for the whole frame (it loads the entry once) and
//     walks the surviving non-blank tokens that its warp is responsible for.  The work per
//     frame scales with the number of surviving tokens (the effect Algorithm 1's pruning is
//     after), and the candidates that get selected - mostly "every entry extended by the
//     frame's dominant token" - sit in different lanes, so they are written side by side.
//   * A candidate that lies above the cut bin of the score histogram is written into the
//     next beam at once by the lane that owns it (slots: stays from the bottom by ballots,
//     extensions from the top by one shared counter per warp and frame).  Only when the cut
//     bin has to be split does a second barrier follow, after which all warps rank the bin's
//     members exactly and write the winners in between; a crowded bin is first split again
//     into 256 sub-bins.
//   * Prefix-trie records are created only for prefixes that are new in the beam and get
//     consecutive node ids; a frame's records leave shared memory with one bulk copy.
//
// Stay candidates, the prefix merge through the table of sequence fingerprints, the score
// histogram with its warp scan, the relative float32 scores with a float64 offset and the
// read-out are those of the general kernel; the two give the same hypotheses and scores that
// agree to float32 rounding.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "fltop_device.cuh"
#include "fltop_internal.h"

namespace fltop {
namespace {

constexpr int kRowCache = 8;     // extension scores a lane keeps in registers per frame
constexpr int kRowsMaxV = 32;    // one token per lane
constexpr unsigned kNoEntry = 0xffffffffu;  // empty table slot; entries are [tag : 20][slot : 12]

__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gmem_src) {
  const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(d), "l"(gmem_src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n"); }
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");
}
__device__ __forceinline__ void cp_async_wait_but_one() {
  asm volatile("cp.async.wait_group 1;\n" ::: "memory");
}
// Asynchronous bulk copy shared -> global (not multicast): block barriers do not wait for it.
__device__ __forceinline__ void bulk_store(void* gmem_dst, const void* smem_src, unsigned bytes) {
  const unsigned s = (unsigned)__cvta_generic_to_shared(smem_src);
  asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;\n" ::"l"(gmem_dst),
               "r"(s), "r"(bytes)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;\n" ::: "memory");
}
__device__ __forceinline__ void bulk_store_wait_read_but_one() {
  asm volatile("cp.async.bulk.wait_group.read 1;\n" ::: "memory");
}
__device__ __forceinline__ void bulk_store_wait_all() {
  asm volatile("cp.async.bulk.wait_group 0;\n" ::: "memory");
}

struct __align__(16) Hot {
  int last;    // last token of the prefix, -1 for the empty prefix
  float pb;    // log-mass of alignments ending in blank (relative)
  float pnb;   // ... ending in the last token
  float tot;   // lse(pb, pnb)
};
struct __align__(16) Ident {
  unsigned long long print;   // fingerprint of the token sequence
  unsigned long long pprint;  // fingerprint of the sequence without its last token
};
struct __align__(8) Where {
  int node;  // trie node of the prefix
  int len;   // its length in tokens
};

// per-frame scalars, one set per frame parity
enum { FS_SLOT_E = 0, FS_WIN_E, FS_LISTN, FS_NSTAY, FS_MAXKEY, FS_COUNT = 8 };  // (the first two: one 8-byte load)
// block scalars
enum { BS_STATUS = 0, BS_CLASHES, BS_NLIVE, BS_EXACT, BS_CNT0, BS_CNT1, BS_CNT2, BS_DEAD, BS_COUNT = 16 };
// What the scan of the score histogram found, as the scanning warp publishes it: everything
// the other warps need, ready to use.
struct __align__(16) CutOut {
  float f_lo;      // a score above this is in the cut bin or above it
  float f_hi;      // a score above this is above the cut bin (= f_lo when the whole bin is kept)
  float best;      // the new zero of the relative scores
  int nbn;         // size of the next beam
  int n_listed;    // members of the cut bin if it has to be split, else 0
  int left;        // how many of them are kept
  int empty;       // 1: no candidate at all
  int thr;         // the cut bin
};

// What every warp has to know about a frame, prepared once by the chore warp a frame ahead.
struct __align__(8) TokLp {
  int tok;     // -1: no such survivor
  float lp;    // -inf then
};
struct __align__(16) FrameHead {
  unsigned kept;     // survivors of the frame (Algorithm 1: top-N stage, conditional break)
  float lp_blank;    // log-probability of blank if it survived, else -inf
  int lg;            // log2 of the lanes a beam entry takes in a row of candidates
  int snb;           // surviving non-blank tokens
};

template <int KMAX>
struct RowsSmem {
  static constexpr int kTable = 16 * KMAX;  // slots of the fingerprint table
  float raw[4][kRowsMaxV];                  // emission rows of frames t .. t+3 as fetched
  Hot hot[2][KMAX];
  Ident ident[2][KMAX];
  Where where[2][KMAX];
  TrieNode nstage[2][KMAX + 2];             // a frame's new trie records
  float st_pb[KMAX], st_pnb[KMAX], st_tot[KMAX];  // the stay candidate of every beam entry
  unsigned dupw[2][KMAX];                   // bit c of word q: "entry q extended by c" is merged
  unsigned tab[2][kTable];
  unsigned hist[kFastBins];
  unsigned hist2[kFastBins];                // the members of a crowded cut bin, binned once more
  int cut2[4];                              // ... and what the scan of that found
  unsigned list_key[kListCap];
  int list_id[kListCap];
  float list_pb[kListCap], list_pnb[kListCap];  // of listed stay candidates
  // the frame as the warps see it: header, the row by token, and by position in a row of
  // candidates the token extended by and its log-probability (-1 / -inf: none)
  // (four copies: a frame is prepared two frames ahead of its use)
  FrameHead head[4];
  float lpv[4][kRowsMaxV];      // by token: its log-probability if it survived, else -inf
  TokLp tokj[4][kRowsMaxV];     // by position among the surviving non-blank tokens
  CutOut cut;
  int fs[2][FS_COUNT];
  int bs[BS_COUNT];
};

// position of the n-th (0-based) set bit of m; m has more than n bits set
__device__ __forceinline__ int nth_set_bit(unsigned m, int n) {
  int pos = 0;
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) {
    const int c = __popc((m >> pos) & ((1u << s) - 1u));
    if (n >= c) { pos += s; n -= c; }
  }
  return pos;
}

// HOOKS bit 0: the survivor mask of every frame is written out (tests); bit 1: the clock at
// every phase boundary is recorded for block 0 (profiling).  Shipped launches use HOOKS = 0.
// BT: SelectTopK's beam_threshold is on - the exact best score of every frame is tracked, and a
// candidate that wins a slot but scores below best - beam_threshold is written as a dead slot
// (probability 0, no identity, not in the table): it yields no candidates and no hypothesis.
template <int MAXT, int MINB, int KMAX, int HOOKS, bool BT>
__global__ void __launch_bounds__(MAXT, MINB) decode_rows_kernel(DecodeParams p) {
  extern __shared__ __align__(16) unsigned char smem_bytes[];
  RowsSmem<KMAX>& S = *reinterpret_cast<RowsSmem<KMAX>*>(smem_bytes);
  constexpr int kTable = RowsSmem<KMAX>::kTable;
  static_assert(KMAX == 64 || KMAX == 128, "the histogram scan takes the bits of K as a template argument");
  constexpr int kBitsOfK = KMAX <= 64 ? 7 : 8;
  const int tid = threadIdx.x, NT = blockDim.x, lane = tid & 31;
  const int b = p.first_wave > 0 ? utterance_by_length(p.lengths, p.B, p.T, p.first_wave,
                                                        reinterpret_cast<int*>(smem_bytes))
                                 : (int)blockIdx.x;
  const int warp = tid >> 5, NW = NT >> 5;
  const int K = p.K, V = p.V, blank = p.blank;
  const unsigned lt_mask = (1u << lane) - 1u;
  const int TS = p.table_slots > 0 ? min(p.table_slots, kTable) : kTable;
  const unsigned tmask = (unsigned)TS - 1u;
  // masses of one prefix are summed, or (merge_max) the larger one is taken: Algorithm 1's
  // literal score' = score + logit, a prefix scores as its best alignment
  const bool use_max = p.merge_max != 0;

  // ---- roles ---------------------------------------------------------------------------
  const int nsw = (K + 31) >> 5;            // stay warps: one lane per beam entry
  const int NXW = NW - 1 - nsw;             // extension warps (at least one)
  const bool is_chore = warp == NW - 1;
  const bool is_stay = warp < nsw;
  const int xw = warp - nsw;                // index among the extension warps
  // An extension warp owns a block of EB beam entries (32, or the beam width rounded up to a
  // power of two when that is less) and, of the surviving tokens, the token rows part,
  // part + P, ...; a token row is 32 / EB tokens wide.
  const int lgE = K >= 32 ? 5 : (K <= 1 ? 0 : 32 - __clz(K - 1));
  const int n_eb = (K + (1 << lgE) - 1) >> lgE;       // entry blocks
  const int P = max(NXW / n_eb, 1);                   // warps that share an entry block
  const int eb = xw % n_eb, part = xw / n_eb;
  const bool is_ext = !is_stay && warp != NW - 1 && part < P;
  const int xq = (eb << lgE) + (lane & ((1 << lgE) - 1));  // this extension lane's beam entry
  const int jsub = lane >> lgE;                       // its token within a token row
  const int lgT = 5 - lgE;                            // log2 of the tokens per token row

  int len = p.lengths[b];
  unsigned flags = 3u;
  if (p.streaming) flags = p.flags ? p.flags[b] : (p.emit_default ? 2u : 0u);
  const bool do_reset = flags & 1u;
  const bool do_emit = (flags & 2u) && p.out_nhyp != nullptr;
  int status = 0;
  bool bad_len = false;
  if (len < 0 || len > p.T) {
    status |= 1;  // FLTOP_ST_BAD_LENGTH
    bad_len = true;
    len = 0;
  }
  TrieNode* const nodes = p.nodes + (int64_t)b * p.nodes_per_utt;
  const int nodes_cap = (int)min(p.nodes_per_utt, (int64_t)0x7ffffff0);
  int32_t* const st = p.streaming
                          ? p.state + (int64_t)b * (kStateHeaderWords + kStateWordsPerSlot * (int64_t)K)
                          : nullptr;

  auto clock_mark = [&](int t, int phase) {
    if ((HOOKS & 2) && b == 0 && lane == 0 && p.dbg_clocks && t >= p.dbg_frame0 &&
        t < p.dbg_frame0 + p.dbg_frames)
      p.dbg_clocks[((int64_t)(t - p.dbg_frame0) * 32 + warp) * 8 + phase] = clock64();
  };

  // ---- initialise shared state ---------------------------------------------------------
  for (int i = tid; i < 2 * KMAX; i += NT) (&S.dupw[0][0])[i] = 0u;
  for (int i = tid; i < 2 * kTable; i += NT) (&S.tab[0][0])[i] = kNoEntry;
  for (int i = tid; i < kFastBins; i += NT) { S.hist[i] = 0u; S.hist2[i] = 0u; }
  if (tid < 2 * FS_COUNT) (&S.fs[0][0])[tid] = 0;
  if (tid < BS_COUNT) S.bs[tid] = 0;
  int cur = 0, nb, n_nodes, frames_seen;
  int created_sum = 0, live_sum = 0, kept_sum = 0, tag_clashes = 0;
  double offset;
  float drift0 = 0.f;  // (streams: carried over from the last chunk)
  if (do_reset) {
    nb = bad_len && !p.streaming ? 0 : 1;
    n_nodes = 2;  // node 0 is the empty prefix, id 1 is not used: a frame's ids start even
    offset = 0.0;
    frames_seen = 0;
    if (tid == 0) {
      Hot e;
      e.last = -1; e.pb = 0.f; e.pnb = neg_inf(); e.tot = 0.f;
      S.hot[0][0] = e;
      S.ident[0][0] = Ident{kRootPrint, 0ull};
      S.where[0][0] = Where{0, 0};
      nodes[0] = TrieNode{-1, -1};
    }
  } else {
    const StateHeader* hd = reinterpret_cast<const StateHeader*>(st);
    nb = hd->nbeam; n_nodes = hd->n_nodes; frames_seen = hd->frames; offset = hd->offset;
    status |= hd->status;
    drift0 = __int_as_float(hd->drift);
    if (!(drift0 <= 0.f && drift0 > -64.f)) drift0 = 0.f;  // (left by another kernel)
    const int32_t* a = st + kStateHeaderWords;
    for (int i = tid; i < nb; i += NT) {
      Hot e;
      e.last = a[K + i];
      e.pb = __int_as_float(a[3 * K + i]);
      e.pnb = __int_as_float(a[4 * K + i]);
      e.tot = __int_as_float(a[5 * K + i]);
      S.hot[0][i] = e;
      S.where[0][i] = Where{a[i], a[2 * K + i]};
      S.ident[0][i] = Ident{reinterpret_cast<const unsigned long long*>(a + 6 * K)[i],
                            reinterpret_cast<const unsigned long long*>(a + 8 * K)[i]};
    }
  }
  __syncthreads();

  // Table of the beam's fingerprints (open addressing, linear probing, at most one slot in
  // sixteen taken).  A probe walk ends at the latest back at its first slot; one that goes all the way
  // round flags the utterance FLTOP_ST_INTERNAL instead of spinning.
  auto table_insert = [&](unsigned* tab, unsigned long long h, int slot) {
    const unsigned val = (((unsigned)h & 0xfffffu) << 12) | (unsigned)slot;
    const unsigned home = (unsigned)(h >> 40) & tmask;
    unsigned pos = home;
    do {
      if (atomicCAS(&tab[pos], kNoEntry, val) == kNoEntry) return;
      pos = (pos + 1) & tmask;
    } while (pos != home);
    atomicOr(&S.bs[BS_STATUS], 16);
  };
  auto table_find = [&](const unsigned* tab, const Ident* ids, unsigned long long h) -> int {
    const unsigned tag = (unsigned)h & 0xfffffu;
    const unsigned home = (unsigned)(h >> 40) & tmask;
    unsigned pos = home;
    do {
      const unsigned v = tab[pos];
      if (v == kNoEntry) return -1;
      if ((v >> 12) == tag) {
        const int slot = (int)(v & 0xfffu);
        if (ids[slot].print == h) return slot;
        ++tag_clashes;
      }
      pos = (pos + 1) & tmask;
    } while (pos != home);
    atomicOr(&S.bs[BS_STATUS], 16);
    return -1;
  };
  for (int i = tid; i < nb; i += NT) table_insert(S.tab[0], S.ident[0][i].print, i);

  // ---- the emission rows: fetched by the chore warp three frames ahead ----------------------
  auto fetch_row = [&](int t1) {
    const int64_t at = (int64_t)b * p.stride_b + (int64_t)t1 * p.stride_t;
    if (p.dtype == kEmissionF32) {
      if (lane < V) cp_async4(&S.raw[t1 & 3][lane], static_cast<const float*>(p.logp) + at + lane);
    } else if (2 * lane < V) {  // two 16-bit emissions per word (V is even then)
      cp_async4(&S.raw[t1 & 3][lane], static_cast<const uint16_t*>(p.logp) + at + 2 * lane);
    }
  };
  // Chore warp: what the warps need to know about frame t1 (its row has landed).  One token
  // per lane: row maximum by a warp reduction, the relative threshold by one float32 add and
  // compare (Algorithm 1's conditional break), the survivors by a ballot.
  // In two halves, so that each fits into a stretch in which the chore warp has nothing else
  // to do: the first ends with the survivor set, the second lays the survivors out.
  float prep_v = neg_inf();   // (chore warp) the row being prepared, one token per lane
  unsigned prep_kept = 0u;    // ... and its survivors
  auto prepare_survivors = [&](int t1) {
    float v = neg_inf();
    if (p.dtype == kEmissionF32) {
      if (lane < V) v = S.raw[t1 & 3][lane];
    } else if (lane < V) {
      const unsigned short bits = reinterpret_cast<const unsigned short*>(S.raw[t1 & 3])[lane];
      v = p.dtype == kEmissionF16 ? __half2float(__ushort_as_half(bits))
                                  : __bfloat162float(__ushort_as_bfloat16(bits));
    }
    // row maximum through an order-preserving integer key (a NaN never is the maximum)
    const unsigned vu = __float_as_uint(v);
    const unsigned vkey = (v == v) ? ((vu & 0x80000000u) ? ~vu : (vu | 0x80000000u)) : 0x007fffffu;
    const unsigned mkey = __reduce_max_sync(kFull, vkey);
    const float m = __uint_as_float((mkey & 0x80000000u) ? (mkey & 0x7fffffffu) : ~mkey);
    const float thr = __fadd_rn(m, p.log_r);
    const bool keep = lane < V && v >= thr;
    unsigned kept = __ballot_sync(kFull, keep);
    if (p.top_n > 0 && __popc(kept) > p.top_n) {
      // stage 1 of Algorithm 1: the best remaining token leaves top_n times (ties: lower id)
      unsigned key = keep ? vkey : 0u;
      unsigned chosen = 0u;
      for (int i = 0; i < p.top_n; ++i) {
        const unsigned best_key = __reduce_max_sync(kFull, key);
        const int w = __ffs(__ballot_sync(kFull, key == best_key)) - 1;
        chosen |= 1u << w;
        if (lane == w) key = 0u;
      }
      kept = chosen;
    }
    prep_v = v;
    prep_kept = kept;
  };
  auto prepare_layout = [&](int t1) {
    const float v = prep_v;
    const unsigned kept = prep_kept;
    const float lb = __shfl_sync(kFull, v, blank);
    const unsigned kept_nb = kept & ~(1u << blank);
    const int snb = __popc(kept_nb);
    const int tok = lane < snb ? nth_set_bit(kept_nb, lane) : -1;
    const float l = __shfl_sync(kFull, v, tok < 0 ? 0 : tok);
    S.lpv[t1 & 3][lane] = ((kept >> lane) & 1u) ? v : neg_inf();
    S.tokj[t1 & 3][lane] = TokLp{tok, tok < 0 ? neg_inf() : l};
    if (lane == 0) {
      FrameHead h;
      h.kept = kept;
      h.lp_blank = ((kept >> blank) & 1u) ? lb : neg_inf();
      h.lg = 0;
      h.snb = snb;
      S.head[t1 & 3] = h;
      kept_sum += __popc(kept);
      if ((HOOKS & 1) && p.dbg_masks) p.dbg_masks[(int64_t)b * p.T + t1] = kept;
    }
  };
  auto prepare = [&](int t1) {
    prepare_survivors(t1);
    prepare_layout(t1);
  };
  if (is_chore) {
    if (len > 0) fetch_row(0);
    if (len > 1) fetch_row(1);
    if (len > 2) fetch_row(2);
    cp_async_commit();
    cp_async_wait_all();
    __syncwarp();
    if (len > 0) prepare(0);
    if (len > 1) prepare(1);
  }
  __syncthreads();

  int pend_at = 0;
  unsigned pend_bytes = 0u;
  const TrieNode* pend_src = S.nstage[0];
  int round = 0;  // block-wide counts taken by the exact fallback so far (its counters rotate)
  int g = 0;      // frames that went through selection so far (its buffers alternate)
  float drift = drift0;  // how far blank-only frames have let the scores sink since
  FrameHead head_next = S.head[0];
  for (int t = 0; t < len; ++t) {
    // the frame as the chore warp prepared it (read before the last barrier of frame t-1)
    const FrameHead head = head_next;
    // Chore warp, while the others evaluate: the trie records of the last selection leave,
    // the row of frame t+3 is requested.
    auto chore_window = [&]() {
      if (lane == 0 && pend_bytes) {
        bulk_store(nodes + pend_at, pend_src, pend_bytes);
        bulk_store_wait_read_but_one();  // the other staging buffer is free again
      }
      if (t + 3 < len) fetch_row(t + 3);
      cp_async_commit();
      cp_async_wait_but_one();  // the row requested a frame ago has landed
      __syncwarp();
      if (t + 2 < len) prepare_survivors(t + 2);
    };
    // A frame in which only blank survives (Algorithm 1's conditional break has dropped every
    // other token): every prefix stays, by blank, and nothing is selected, merged or created.
    // The beam is updated where it is; the scores sink a little, which the next ordinary frame
    // takes back into the offset (a long run of such frames is cut short by one).
    if (head.snb == 0 && ((head.kept >> blank) & 1u) && drift > -6.f) {
      if (is_stay && tid < nb) {
        Hot e = S.hot[cur][tid];
        e.pb = e.tot + head.lp_blank;
        e.pnb = neg_inf();
        e.tot = e.pb;
        S.hot[cur][tid] = e;
      } else if (is_chore) {
        chore_window();
        if (t + 2 < len) prepare_layout(t + 2);
      }
      if (BT && is_stay) {  // dead slots stay dead and are not counted as held prefixes
        const unsigned dead = __ballot_sync(kFull, tid < nb && S.hot[cur][tid].tot == neg_inf());
        if (lane == 0 && dead) atomicAdd(&S.bs[BS_DEAD], __popc(dead));
      }
      drift += head.lp_blank;
      pend_bytes = 0u;
      live_sum += nb;
      head_next = S.head[(t + 1) & 3];  // prepared a frame ago
      __syncthreads();
      continue;
    }
    drift = 0.f;
    const int par = g & 1, nxt = cur ^ 1;
    ++g;
    const Hot* const hc = S.hot[cur];
    Hot* const hn = S.hot[nxt];
    const Ident* const id_c = S.ident[cur];
    Ident* const id_n = S.ident[nxt];
    const Where* const wh_c = S.where[cur];
    Where* const wh_n = S.where[nxt];
    unsigned* const hist = S.hist;
    unsigned* const dupw = S.dupw[par];
    const unsigned* const tab_c = S.tab[cur];
    unsigned* const tab_n = S.tab[nxt];
    int* const fs = S.fs[par];
    TrieNode* const nst = S.nstage[par];
    clock_mark(t, 0);

    const TokLp* const tokj = S.tokj[t & 3];
    const int n_trows = (head.snb + (1 << lgT) - 1) >> lgT;  // token rows of this frame
    // position (among the surviving non-blank tokens) of the token of this lane's k-th row
    auto row_token = [&](int k) -> int { return ((part + k * P) << lgT) + jsub; };
    // (with few survivors most extension warps have no row at all and sit the frame out)
    const bool has_rows = is_ext && part < n_trows;

    // ---- P1: every candidate is evaluated once and counted ---------------------------------
    // Extension lanes keep the scores of their first rows in registers, and what their best
    // candidate needs to be written into the next beam: while the stay warps are still busy
    // (theirs is the longer chain) they work out its token and its fingerprint.
    float kc[kRowCache];
#pragma unroll
    for (int k = 0; k < kRowCache; ++k) kc[k] = neg_inf();
    float far_max = neg_inf();               // (BT) best score among the rows beyond the cache
    float sc1 = neg_inf(), sc2 = neg_inf();  // best and second-best cached score of this lane
    int j1 = 0, tok1 = 0;                    // position and token of the best
    unsigned long long hp = 0ull, h1 = 0ull; // fingerprints of the entry and of the best candidate
    Where xwh = Where{0, 0};
    // the beam entry of this lane (stay lanes: entry tid; extension lanes: entry xq)
    Hot se;
    se.last = -1; se.pb = se.pnb = se.tot = neg_inf();
    // stay lanes: identity and stay candidate stay in registers until they are placed
    Ident sid = Ident{0ull, 0ull};
    Where swh = Where{0, 0};
    float npb = neg_inf(), npnb = neg_inf(), stot = neg_inf();
    float s_own = neg_inf(), s_dup = neg_inf();
    float other_tot[KMAX / 32];  // the stay candidates of lane `lane` of every stay warp
#pragma unroll
    for (int w = 0; w < KMAX / 32; ++w) other_tot[w] = neg_inf();
    if (is_stay) {
      if (tid < nb) {
        se = hc[tid];
        sid = id_c[tid];
        npb = se.tot + head.lp_blank;
        float own = neg_inf(), dup = neg_inf();
        if (se.last >= 0) {
          const float le = S.lpv[t & 3][se.last];  // -inf if the token did not survive
          own = se.pnb + le;
          const int pq = table_find(tab_c, id_c, sid.pprint);
          if (pq >= 0) {
            const Hot pe = hc[pq];
            dup = ((pe.last == se.last) ? pe.pb : pe.tot) + le;
            if (dup != neg_inf()) {  // the parent's extension by last(q) names this prefix
              atomicSub(&hist[score_bin(dup)], 1u);
              atomicOr(&dupw[pq], 1u << se.last);
            }
          }
        }
        stot = use_max ? fmaxf(npb, fmaxf(own, dup)) : lse3(npb, own, dup);
        if (stot != neg_inf()) atomicAdd(&hist[score_bin(stot)], 1u);
        s_own = own;
        s_dup = dup;
      }
      if (tid < KMAX) S.st_tot[tid] = stot;
    } else if (has_rows) {
      if (xq < nb) {
        se = hc[xq];
        hp = id_c[xq].print;
        xwh = wh_c[xq];
      }
      // (a position past the last survivor holds token -1 and log-probability -inf)
#pragma unroll
      for (int k = 0; k < kRowCache; ++k) {
        if (part + k * P >= n_trows) break;
        const int j = row_token(k);
        const TokLp tl = tokj[j];
        const float sc = ((tl.tok == se.last) ? se.pb : se.tot) + tl.lp;
        kc[k] = sc;
        if (sc != neg_inf()) atomicAdd(&hist[score_bin(sc)], 1u);
        const bool better = sc > sc1;
        sc2 = better ? sc1 : fmaxf(sc2, sc);
        j1 = better ? j : j1;
        sc1 = better ? sc : sc1;
      }
#pragma unroll 1
      for (int k = kRowCache; part + k * P < n_trows; ++k) {  // evaluated again later
        const TokLp tl = tokj[row_token(k)];
        const float sc = ((tl.tok == se.last) ? se.pb : se.tot) + tl.lp;
        if (sc != neg_inf()) atomicAdd(&hist[score_bin(sc)], 1u);
        if (BT) far_max = fmaxf(far_max, sc);
      }
      tok1 = tokj[j1].tok;
      if (sc1 != neg_inf()) h1 = child_print(hp, tok1);
    } else if (is_chore) {
      chore_window();
    }
    clock_mark(t, 1);
    __syncthreads();  // B1: the histogram is complete
    clock_mark(t, 2);

    // ---- P2: the chore warp scans the histogram; the others meanwhile empty the table that
    // the next beam's fingerprints go into
    if (is_chore) {
      const Cut c = scan_score_histogram_ballots<kBitsOfK>(hist, K);
      if (lane == 0) {
        CutOut o;
        const bool all = c.cut_count == c.left;  // also true when there is no cut at all
        o.f_lo = (c.thr >= kFastBins - 1) ? neg_inf() : -(float)(c.thr + 1) * (1.f / kBinsPerNat);
        o.f_hi = all ? o.f_lo
                     : (c.thr == 0 ? __int_as_float(0x7f800000) : -(float)c.thr * (1.f / kBinsPerNat));
        // new zero of the relative scores: the upper edge of the first non-empty group of bins
        o.best = -(float)(c.first * kBinsPerLane) * (1.f / kBinsPerNat);
        o.nbn = min(c.total, K);
        o.n_listed = all ? 0 : c.cut_count;
        o.left = c.left;
        o.empty = c.total == 0 ? 1 : 0;
        o.thr = c.thr;
        S.cut = o;

      }
    } else {
      if (is_stay) {
        const uint4 ones = make_uint4(~0u, ~0u, ~0u, ~0u);
        uint4* const t_n = reinterpret_cast<uint4*>(tab_n);
        for (int i = tid; i < kTable / 4; i += 32 * nsw) t_n[i] = ones;
        // what a stay candidate needs only if it is kept, and the other stay warps'
        // candidates: fetched and worked out while the scan runs
        if (tid < nb) {
          npnb = use_max ? fmaxf(s_own, s_dup) : lse2(s_own, s_dup);
          swh = wh_c[tid];
        }
#pragma unroll
        for (int w = 0; w < KMAX / 32; ++w) other_tot[w] = (w < nsw) ? S.st_tot[w * 32 + lane] : neg_inf();
      } else if (is_ext && sc1 != neg_inf()) {
        // an extension that a stay candidate has absorbed (the merge) is no candidate
        if ((dupw[xq] >> tok1) & 1u) sc1 = neg_inf();
      }
    }
    clock_mark(t, 3);
    __syncthreads();  // B2: the cut is known
    const CutOut cut = S.cut;
    const float best = cut.best, f_lo = cut.f_lo, f_hi = cut.f_hi;
    int n_listed = cut.n_listed, left = cut.left;
    const int nbn = cut.nbn;
    const bool arena_ok = n_nodes + ((K + 1) & ~1) <= nodes_cap;
    // (BT) SelectTopK's beam_threshold: kept scores reach the frame's exact best minus the
    // threshold.  No score lies above the reference edge by more than log 3 (a stay candidate
    // sums three masses that are each below it), so when even the lower edge of the cut bin
    // is within the threshold of that bound nothing can be dropped and the exact best is not
    // needed; otherwise the block reduces it (one more barrier).
    float floor_sc = neg_inf();
    if (BT && f_lo < best + 2.f - p.beam_threshold) {  // block-uniform
      if (is_stay || has_rows) {
        // (an absorbed extension never beats the stay candidate it went into)
        const unsigned key = __reduce_max_sync(kFull, score_key(is_stay ? stot : fmaxf(sc1, far_max)));
        if (lane == 0 && key) atomicMax(reinterpret_cast<unsigned*>(&fs[FS_MAXKEY]), key);
      }
      __syncthreads();
      const unsigned mk = (unsigned)fs[FS_MAXKEY];
      if (mk) floor_sc = key_score(mk) - p.beam_threshold;
    }

    // A crowded cut bin (more members than the pairwise ranking takes) is binned once more:
    // an inner bin into 256 sub-bins over its quarter nat, the last bin - everything more
    // than 63.75 nats below the reference, where the hopeless candidates of a sharply peaked
    // utterance collect - into quarter-nat bins over the next 64 nats.  The cut is then
    // located among those and only that sub-bin's members are ranked.
    const bool refined = n_listed > kListCap;  // block-uniform
    const float hi_edge = -(float)cut.thr * (1.f / kBinsPerNat);
    const float sub_scale = cut.thr >= kFastBins - 1 ? kBinsPerNat : kBinsPerNat * (float)kFastBins;
    int sub_thr = 0;
    bool sub_all = false;
    auto sub_bin = [&](float sc) -> int {
      const int b2 = __float2int_rz((hi_edge - sc) * sub_scale);
      return min(kFastBins - 1, max(0, b2));
    };
    // 2: the candidate is kept, 1: it is in the (sub-)bin that the cut runs through, 0: it is out
    auto klass = [&](float sc) -> int {
      if (sc > f_hi) return 2;
      if (!(sc > f_lo)) return 0;
      if (!refined) return 1;
      const int sb = sub_bin(sc);
      return sb < sub_thr ? 2 : (sb == sub_thr ? (sub_all ? 2 : 1) : 0);
    };
    if (refined) {
      auto count2 = [&](float sc) {
        if (sc > f_lo && !(sc > f_hi)) atomicAdd(&S.hist2[sub_bin(sc)], 1u);
      };
      if (is_stay) {
        count2(stot);
      } else if (is_ext && xq < nb) {
        const unsigned dw = dupw[xq];
#pragma unroll 1
        for (int k = 0; part + k * P < n_trows; ++k) {
          const TokLp tl = tokj[row_token(k)];
          if (tl.tok >= 0 && !((dw >> tl.tok) & 1u))
            count2(((tl.tok == se.last) ? se.pb : se.tot) + tl.lp);
        }
      }
      __syncthreads();
      if (is_chore) {
        const Cut c2 = scan_score_histogram_ballots<kBitsOfK>(S.hist2, left);
        if (lane == 0) {
          S.cut2[0] = c2.thr; S.cut2[1] = c2.left; S.cut2[2] = c2.cut_count;
          S.cut2[3] = c2.cut_count == c2.left ? 1 : 0;
        }
        __syncwarp();
        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
        reinterpret_cast<uint4*>(S.hist2)[lane] = zero;
        reinterpret_cast<uint4*>(S.hist2)[lane + 32] = zero;
      }
      __syncthreads();
      sub_thr = S.cut2[0];
      sub_all = S.cut2[3] != 0;
      left = S.cut2[1];
      n_listed = sub_all ? 0 : S.cut2[2];
    }
    if ((HOOKS & 2) && b == 0 && tid == 0 && p.dbg_clocks && t >= p.dbg_frame0 &&
        t < p.dbg_frame0 + p.dbg_frames) {
      // (rows 24.. of the record are free: fewer than 24 warps) what the scan found
      long long* const o = p.dbg_clocks + ((int64_t)(t - p.dbg_frame0) * 32 + 24) * 8;
      o[0] = nbn; o[1] = n_listed; o[2] = left; o[3] = cut.empty; o[4] = nb;
      o[5] = head.snb; o[6] = n_trows; o[7] = 0;
    }

    // writing candidates into the next beam
    auto place_dead = [&](int slot) {
      Hot e;
      e.last = -1; e.pb = e.pnb = e.tot = neg_inf();
      hn[slot] = e;
      id_n[slot] = Ident{0ull, 0ull};
      wh_n[slot] = Where{0, 0};
      atomicAdd(&S.bs[BS_DEAD], 1);
    };
    auto place_stay_from = [&](int q, float pb_q, float pnb_q, float tot_q, int slot) {
      if ((unsigned)slot >= (unsigned)K) return;  // only reachable with NaN scores
      if (BT && tot_q < floor_sc) return place_dead(slot);
      Hot e;
      e.last = hc[q].last; e.pb = pb_q - best; e.pnb = pnb_q - best; e.tot = tot_q - best;
      hn[slot] = e;
      const Ident id = id_c[q];
      id_n[slot] = id;
      wh_n[slot] = wh_c[q];
      table_insert(tab_n, id.print, slot);
    };
    // a new prefix: entry q (fingerprint hp_q, trie place w_q) extended by tok, fingerprint h;
    // `ord` numbers the frame's new prefixes
    auto place_new = [&](unsigned long long hp_q, Where w_q, int tok, unsigned long long h,
                         float sc, int slot, int ord) {
      if ((unsigned)slot >= (unsigned)K || (unsigned)ord >= (unsigned)K) return;
      nst[ord] = TrieNode{w_q.node, tok};  // (also for a dead slot: the frame's records are one run)
      if (BT && sc < floor_sc) return place_dead(slot);
      Hot e;
      e.last = tok; e.pb = neg_inf(); e.pnb = sc - best; e.tot = sc - best;
      hn[slot] = e;
      id_n[slot] = Ident{h, hp_q};
      wh_n[slot] = Where{arena_ok ? n_nodes + ord : 0, w_q.len + 1};
      table_insert(tab_n, h, slot);
    };
    auto place_ext = [&](int q, int tok, float sc, int slot, int ord) {
      const unsigned long long hp_q = id_c[q].print;
      place_new(hp_q, wh_c[q], tok, child_print(hp_q, tok), sc, slot, ord);
    };
    // lanes with `want` take consecutive places from a counter: one update for the warp
    auto take_places = [&](bool want, int* counter) -> int {
      const unsigned m = __ballot_sync(kFull, want);
      if (!m) return 0;
      int base = 0;
      if (lane == 0) base = atomicAdd(counter, __popc(m));
      return __shfl_sync(kFull, base, 0) + __popc(m & lt_mask);
    };
    auto list_add = [&](int at, float sc, int id) {
      if (at < kListCap) {
        S.list_key[at] = score_key(sc);
        S.list_id[at] = id;
      }
    };
    // chore warp, once the cut is out: the histogram and the counters and merge bits of frame
    // t+1 start empty (nobody touches any of them before B4)
    auto chore_after_cut = [&]() {
      const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
      reinterpret_cast<uint4*>(hist)[lane] = zero;
      reinterpret_cast<uint4*>(hist)[lane + 32] = zero;
      if (lane < KMAX / 4) reinterpret_cast<uint4*>(S.dupw[par ^ 1])[lane] = zero;
      if (lane < FS_COUNT) S.fs[par ^ 1][lane] = 0;
      // frame t+2 as the warps will see it (the buffers it goes into were last read in
      // frame t-2); the survivor set was worked out while the others evaluated
      if (t + 2 < len) prepare_layout(t + 2);
    };

    if (n_listed <= kListCap) {
      // ---- P3: candidates above the cut bin take their slots and are written at once -------
      if (is_stay) {
        // every stay warp looks at all stay candidates itself: the slots follow from ballots
        int before = 0, total_sel = 0;
        int kl = 0;
        unsigned m_own = 0u;
#pragma unroll
        for (int w = 0; w < KMAX / 32; ++w) {
          if (w < nsw) {
            const int k_w = klass(other_tot[w]);
            const unsigned m_w = __ballot_sync(kFull, k_w == 2);
            const int n_w = __popc(m_w);
            before += w < warp ? n_w : 0;
            total_sel += n_w;
            if (w == warp) { kl = k_w; m_own = m_w; }
          }
        }
        if (tid == 0) fs[FS_NSTAY] = total_sel;
        if (kl == 2) {
          const int slot = before + __popc(m_own & lt_mask);
          if (BT && (unsigned)slot < (unsigned)K && stot < floor_sc) {
            place_dead(slot);
          } else if ((unsigned)slot < (unsigned)K) {
            Hot e;
            e.last = se.last; e.pb = npb - best; e.pnb = npnb - best; e.tot = stot - best;
            hn[slot] = e;
            id_n[slot] = sid;
            wh_n[slot] = swh;
            table_insert(tab_n, sid.print, slot);
          }
        }
        if (n_listed > 0) {
          const int at = take_places(kl == 1, &fs[FS_LISTN]);
          if (kl == 1 && at < kListCap) {
            list_add(at, stot, tid << 16);
            S.list_pb[at] = npb;
            S.list_pnb[at] = npnb;
          }
        }
      } else if (has_rows) {
        // this lane's best candidate first (its token and fingerprint are ready) ...
        const int kl1 = klass(sc1);
        const bool in1 = kl1 != 0;
        if (__any_sync(kFull, in1 || sc2 > f_lo)) {
          const bool sure1 = kl1 == 2;
          const int ord = take_places(sure1, &fs[FS_SLOT_E]);
          if (sure1) place_new(hp, xwh, tok1, h1, sc1, nbn - 1 - ord, ord);
          if (n_listed > 0) {
            const int at = take_places(in1 && !sure1, &fs[FS_LISTN]);
            if (in1 && !sure1) list_add(at, sc1, (xq << 16) | (tok1 + 1));
          }
          // ... then, if a lane has more than one (a frame with competing tokens), the others
          if (__any_sync(kFull, sc2 > f_lo)) {
            unsigned sure = 0u, lst = 0u;
            if (sc2 > f_lo) {
              const unsigned dw = dupw[xq];
#pragma unroll
              for (int k = 0; k < kRowCache; ++k) {
                if (kc[k] > f_lo && row_token(k) != j1 && !((dw >> tokj[row_token(k)].tok) & 1u)) {
                  const int kl = klass(kc[k]);
                  if (kl == 2) sure |= 1u << k;
                  else if (kl == 1) lst |= 1u << k;
                }
              }
            }
            // the cached score of row k (k differs from lane to lane)
            auto cached = [&](int k) -> float {
              float v = kc[0];
#pragma unroll
              for (int i = 1; i < kRowCache; ++i) v = (k == i) ? kc[i] : v;
              return v;
            };
            while (__any_sync(kFull, sure != 0u)) {  // one candidate per lane and round
              const int ord2 = take_places(sure != 0u, &fs[FS_SLOT_E]);
              if (sure) {
                const int k = __ffs(sure) - 1;
                sure &= sure - 1;
                place_ext(xq, tokj[row_token(k)].tok, cached(k), nbn - 1 - ord2, ord2);
              }
            }
            while (n_listed > 0 && __any_sync(kFull, lst != 0u)) {
              const int at = take_places(lst != 0u, &fs[FS_LISTN]);
              if (lst) {
                const int k = __ffs(lst) - 1;
                lst &= lst - 1;
                list_add(at, cached(k), (xq << 16) | (tokj[row_token(k)].tok + 1));
              }
            }
          }
        }
        // rows beyond the cache: evaluated again, a counter update per row
#pragma unroll 1
        for (int k = kRowCache; part + k * P < n_trows; ++k) {
          const TokLp tl = tokj[row_token(k)];
          const int tok = tl.tok;
          float sc = ((tok == se.last) ? se.pb : se.tot) + tl.lp;
          if (sc > f_lo && ((dupw[xq] >> tok) & 1u)) sc = neg_inf();
          const int kl = klass(sc);
          const bool isin = kl != 0, issure = kl == 2;
          if (__any_sync(kFull, isin)) {
            const int ord = take_places(issure, &fs[FS_SLOT_E]);
            if (issure) place_ext(xq, tok, sc, nbn - 1 - ord, ord);
            if (n_listed > 0) {
              const int at = take_places(isin && !issure, &fs[FS_LISTN]);
              if (isin && !issure) list_add(at, sc, (xq << 16) | (tok + 1));
            }
          }
        }
      } else if (is_chore) {
        chore_after_cut();
      }
      clock_mark(t, 4);
      if (n_listed > 0) {  // block-uniform
        __syncthreads();   // B3: the members of the cut bin are listed
        clock_mark(t, 5);
        // The members of the cut bin are ranked by (score, candidate id) and the best `left`
        // go to the slots between the stays and the extensions.  All warps share the work: a
        // warp takes every NW-th member and counts, with one ballot per 32 members, how many
        // beat it; then one lane per winner writes it.
        const int n = min(fs[FS_LISTN], kListCap);
        const int n_stay = min(fs[FS_NSTAY], K), n_ext = fs[FS_SLOT_E];
        const unsigned key_a = lane < n ? S.list_key[lane] : 0u;
        const int id_a = lane < n ? S.list_id[lane] : 0;
        const unsigned key_b = lane + 32 < n ? S.list_key[lane + 32] : 0u;
        const int id_b = lane + 32 < n ? S.list_id[lane + 32] : 0;
        int n_won = 0, my_m = -1, my_rank = 0;
#pragma unroll 1
        for (int m = warp; m < n; m += NW) {
          const unsigned key = S.list_key[m];
          const int id = S.list_id[m];
          int rank = __popc(__ballot_sync(
              kFull, lane < n && (key_a > key || (key_a == key && id_a < id))));
          if (n > 32)
            rank += __popc(__ballot_sync(
                kFull, lane + 32 < n && (key_b > key || (key_b == key && id_b < id))));
          if (rank < left) {
            if (lane == n_won) { my_m = m; my_rank = rank; }
            ++n_won;
          }
        }
        if (n_won) {  // warp-uniform; lane i writes the i-th winner this warp found
          const bool mine = my_m >= 0;
          const int id = mine ? S.list_id[my_m] : 0;
          const bool new_prefix = mine && (id & 0xffff) != 0;
          const int ord = n_ext + take_places(new_prefix, &fs[FS_WIN_E]);
          if (mine) {
            const int q = id >> 16, slot = n_stay + my_rank;
            const float sc = key_score(S.list_key[my_m]);
            if (new_prefix) place_ext(q, (id & 0xffff) - 1, sc, slot, ord);
            else place_stay_from(q, S.list_pb[my_m], S.list_pnb[my_m], sc, slot);
          }
        }
      }
    } else {
      // ---- exact fallback: the cut bin holds more members than the pairwise ranking takes.
      // The K-th best key is found bit by bit (a block-wide count per bit), then, among the
      // candidates that share it, the id of the last one that still fits; every candidate then
      // knows by itself whether it is in.  Slow (some sixty barriers) and rare: rows of nearly
      // equal probabilities.
      if (is_chore) chore_after_cut();
      auto for_each_candidate = [&](auto&& f) {
        if (is_stay) {
          if (tid < nb) f(score_key(stot), tid << 16);
        } else if (is_ext && xq < nb) {
          const unsigned dw = dupw[xq];
#pragma unroll 1
          for (int k = 0; part + k * P < n_trows; ++k) {
            const TokLp tl = tokj[row_token(k)];
            const int tok = tl.tok;
            if (tok < 0) continue;
            const float sc = ((tok == se.last) ? se.pb : se.tot) + tl.lp;
            unsigned key = score_key(sc);
            if ((dw >> tok) & 1u) key = 0u;
            f(key, (xq << 16) | (tok + 1));
          }
        }
      };
      // number of candidates for which pred holds (block-uniform result)
      auto block_count = [&](auto&& pred) -> int {
        int mine = 0;
        for_each_candidate([&](unsigned key, int id) { mine += (key && pred(key, id)) ? 1 : 0; });
        mine = __reduce_add_sync(kFull, mine);
        int* const cnt = &S.bs[BS_CNT0 + round % 3];
        if (lane == 0 && mine) atomicAdd(cnt, mine);
        if (tid == 0) S.bs[BS_CNT0 + (round + 1) % 3] = 0;  // last read two barriers ago
        __syncthreads();
        ++round;
        return *cnt;
      };
      unsigned kth = 0u;
#pragma unroll 1
      for (int bit = 31; bit >= 0; --bit) {
        const unsigned trial = kth | (1u << bit);
        if (block_count([&](unsigned key, int) { return key >= trial; }) >= K) kth = trial;
      }
      const int n_gt = block_count([&](unsigned key, int) { return key > kth; });
      const int need = K - n_gt;  // how many of the candidates with the K-th key fit (>= 1)
      // the need-th smallest id among them, bit by bit from the top (ids are below 2^23)
      int id_cut = 0;
#pragma unroll 1
      for (int bit = 22; bit >= 0; --bit) {
        const int trial = id_cut | (1 << bit);
        // ids below `trial`: if fewer than `need`, the id we look for is at least `trial`
        if (block_count([&](unsigned key, int id) { return key == kth && id < trial; }) < need)
          id_cut = trial;
      }
      // slots: one counter for all (the order inside the beam carries no meaning)
      for_each_candidate([&](unsigned key, int id) {
        if (!key || !(key > kth || (key == kth && id <= id_cut))) return;
        const int q = id >> 16;
        if ((id & 0xffff) == 0) {
          const int slot = atomicAdd(&fs[FS_NSTAY], 1);
          place_stay_from(q, npb, npnb, stot, slot);
        } else {
          const int ord = atomicAdd(&fs[FS_SLOT_E], 1);
          place_ext(q, (id & 0xffff) - 1, key_score(key), nbn - 1 - ord, ord);
        }
      });
      if (tid == 0) atomicAdd(&S.bs[BS_EXACT], 1);
    }

    if (cut.empty) status |= 8;  // FLTOP_ST_EMPTY_BEAM
    if (is_stay) offset += (double)best;  // (the stay lanes write the scores out)
    clock_mark(t, 6);
    head_next = S.head[(t + 1) & 3];  // prepared a frame ago
    __syncthreads();  // B4: the next beam and its table are complete
    clock_mark(t, 7);

    const int2 new2 = *reinterpret_cast<const int2*>(&fs[FS_SLOT_E]);
    const int made = new2.x + new2.y;  // new prefixes of this frame
    pend_at = n_nodes;
    pend_src = nst;
    pend_bytes = (arena_ok && made > 0) ? (unsigned)(((made + 1) & ~1) * sizeof(TrieNode)) : 0u;
    if (!arena_ok && made > 0) status |= 2;  // FLTOP_ST_ARENA_FULL
    if (arena_ok) n_nodes += (made + 1) & ~1;
    created_sum += made;
    live_sum += nbn;
    nb = nbn;
    cur = nxt;
  }
  frames_seen += len;
  // (survivors are not listed per frame: their total goes out with the statistics)
  if (p.stats && is_chore && lane == 0) p.stats[kStatWords * (int64_t)b + 6] = kept_sum;
  // the last frame's records; the read-out below walks the trie, so wait for all of them
  if (is_chore && lane == 0) {
    if (pend_bytes) bulk_store(nodes + pend_at, pend_src, pend_bytes);
    bulk_store_wait_all();
  }
  if (tag_clashes) atomicAdd(&S.bs[BS_CLASHES], tag_clashes);
  __syncthreads();

  status |= S.bs[BS_STATUS];
  if (p.stats && tid == 0) {
    int32_t* o = p.stats + kStatWords * (int64_t)b;
    o[0] = len; o[1] = created_sum; o[2] = live_sum - S.bs[BS_DEAD]; o[3] = n_nodes;
    o[4] = S.bs[BS_CLASHES]; o[5] = S.bs[BS_EXACT];
  }

  const Hot* const hc = S.hot[cur];
  const Ident* const id_c = S.ident[cur];
  const Where* const wh_c = S.where[cur];

  // ---- keep the beam for the next chunk (streaming) ---------------------------------------
  if (p.streaming) {
    int32_t* a = st + kStateHeaderWords;
    for (int i = tid; i < nb; i += NT) {
      const Hot e = hc[i];
      const Where w = wh_c[i];
      const Ident id = id_c[i];
      a[i] = w.node; a[K + i] = e.last; a[2 * K + i] = w.len;
      a[3 * K + i] = __float_as_int(e.pb); a[4 * K + i] = __float_as_int(e.pnb);
      a[5 * K + i] = __float_as_int(e.tot);
      reinterpret_cast<unsigned long long*>(a + 6 * K)[i] = id.print;
      reinterpret_cast<unsigned long long*>(a + 8 * K)[i] = id.pprint;
    }
    if (tid == 0) {
      StateHeader* hd = reinterpret_cast<StateHeader*>(st);
      hd->nbeam = nb; hd->n_nodes = n_nodes; hd->frames = frames_seen;
      hd->status = status & ~1;  // a bad chunk length is not sticky
      hd->offset = offset;
      hd->drift = __float_as_int(drift);
    }
  }

  // ---- hypotheses, best first (GetHighestScorePrefix over the whole beam) -----------------
  if (do_emit) {
    const int Lout = p.L;
    bool truncated = false;
    for (int i = tid; i < nb; i += NT) {
      const float ti = hc[i].tot;
      if (ti == neg_inf()) continue;
      atomicAdd(&S.bs[BS_NLIVE], 1);
      int rank = 0;
      for (int j = 0; j < nb; ++j) {
        const float tj = hc[j].tot;
        rank += (tj > ti || (tj == ti && j < i)) ? 1 : 0;
      }
      const int64_t o = (int64_t)b * K + rank;
      p.out_scores[o] = (float)(offset + (double)ti);
      const Where w = wh_c[i];
      const int n = w.len;
      p.out_lens[o] = n;
      if (n > Lout) truncated = true;
      int32_t* dst = p.out_tokens + o * Lout;
      int node = w.node;
      for (int d = n - 1; d >= 0 && node > 0 && (int64_t)node < p.nodes_per_utt; --d) {
        const int2 rec = *reinterpret_cast<const int2*>(&nodes[node]);  // parent, token
        if (d < Lout) dst[d] = rec.y;
        node = rec.x;
      }
    }
    if (truncated) atomicOr(&S.bs[BS_STATUS], 4);  // FLTOP_ST_TRUNCATED
    __syncthreads();
    const int n_live = S.bs[BS_NLIVE];
    for (int k = n_live + tid; k < K; k += NT) {
      p.out_lens[(int64_t)b * K + k] = 0;
      p.out_scores[(int64_t)b * K + k] = neg_inf();
    }
    status |= S.bs[BS_STATUS];
    if (tid == 0) p.out_nhyp[b] = n_live;
  }
  if (tid == 0 && p.out_status) p.out_status[b] = status;
}

constexpr int kRowsKmax = 128;  // widest beam; beams up to 64 have an instantiation of their own

template <int HOOKS, int KMAX, bool BT = false>
cudaError_t launch_rows_hooks(const DecodeParams& p0, int nt, bool alone, int sms, cudaStream_t s) {
  const size_t bytes = sizeof(RowsSmem<KMAX>);
  void (*kernel)(DecodeParams) = (alone && nt <= 512) ? decode_rows_kernel<512, 1, KMAX, HOOKS, BT>
                                                      : decode_rows_kernel<1024, 1, KMAX, HOOKS, BT>;
  static_assert(sizeof(RowsSmem<KMAX>) <= 48 * 1024, "fits without the opt-in attribute");
  DecodeParams p = p0;
  if (p.first_wave > 0) {
    // blocks that do not all fit on the GPU at once start longest first throughout
    int per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, nt, bytes) != cudaSuccess) {
      cudaGetLastError();
      per_sm = 1;
    }
    p.first_wave = (int64_t)p.B <= (int64_t)per_sm * sms ? sms : p.B;
  }
  kernel<<<p.B, nt, bytes, s>>>(p);
  return cudaGetLastError();
}

}  // namespace

bool decode_rows_eligible(const DecodeParams& p) {
  // (the instrumented instantiations exist without beam_threshold only)
  const bool hooked = p.dbg_masks != nullptr || p.dbg_clocks != nullptr;
  return p.K <= kRowsKmax && p.V <= kRowsMaxV && p.logp != nullptr &&
         !(p.beam_threshold > 0.f && hooked);
}

// Threads per block: the stay warps, the chore warp, and for every block of 32 beam entries P
// extension warps that share the frame's surviving tokens among them.
int decode_rows_threads(const DecodeParams& p, bool alone) {
  const int nsw = (p.K + 31) / 32;
  int cols = p.V - 1;  // non-blank survivors of a frame, as far as the host can tell
  if (p.pruning) cols = cols > 12 ? 12 : cols;
  if (p.top_n > 0 && p.top_n < cols) cols = p.top_n;
  const int per_row = p.K >= 32 ? 1 : 32 / (p.K <= 1 ? 1 : 1 << (32 - __builtin_clz(p.K - 1)));
  const int rows = (cols + per_row - 1) / per_row;   // token rows of a frame
  // measured on B200 (64 utterances, V = 32): with pruning on four warps per block of beam
  // entries for beams above 32, six below; without, as many as fit; a quarter of that when
  // blocks share SMs
  int P = alone ? (rows + 1) / 2 : (rows + 3) / 4;
  const int cap = ((alone ? 16 : 8) - 1 - nsw) / nsw;
  if (alone && p.pruning && nsw > 1 && P > 4) P = 4;
  if (P > cap) P = cap;
  // beams above 96 without pruning: four warps per block of entries (21 warps) beat the cap's two
  // (K = 100, r = 0: 4.8 against 6.1 ms)
  if (alone && !p.pruning && nsw >= 4 && rows >= 8) P = 4;
  if (P < 1) P = 1;
  return 32 * (nsw + 1 + nsw * P);
}

cudaError_t launch_decode_rows(const DecodeParams& p, cudaStream_t s) {
  if (p.B == 0) return cudaSuccess;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int blocks = p.co_resident > p.B ? p.co_resident : p.B;
  const bool alone = blocks <= sms;
  const int nsw = (p.K + 31) / 32;
  int nt = p.block_threads > 0 ? p.block_threads : decode_rows_threads(p, alone);
  nt = (nt + 31) / 32 * 32;
  if (nt < 32 * (2 * nsw + 1)) nt = 32 * (2 * nsw + 1);  // stay warps, as many extension warps, the chore warp
  if (nt > kMaxThreads) nt = kMaxThreads;
  const int hooks = (p.dbg_masks ? 1 : 0) | (p.dbg_clocks ? 2 : 0);
  DecodeParams q = p;
  // more utterances of one batch than SMs: the blocks take them by length
  q.first_wave = (!p.streaming && p.co_resident == 0 && p.B > sms && p.B <= kByLengthMaxB) ? sms : 0;
  static_assert(sizeof(RowsSmem<64>) >= (kByLengthMaxB + 1) * sizeof(int), "scratch of the ranking");
  if (p.beam_threshold > 0.f) {
    return p.K <= 64 ? launch_rows_hooks<0, 64, true>(q, nt, alone, sms, s)
                     : launch_rows_hooks<0, 128, true>(q, nt, alone, sms, s);
  }
  if (p.K <= 64) {
    switch (hooks) {
      case 0: return launch_rows_hooks<0, 64>(q, nt, alone, sms, s);
      case 1: return launch_rows_hooks<1, 64>(q, nt, alone, sms, s);
      default: return launch_rows_hooks<3, 64>(q, nt, alone, sms, s);
    }
  }
  switch (hooks) {
    case 0: return launch_rows_hooks<0, 128>(q, nt, alone, sms, s);
    case 1: return launch_rows_hooks<1, 128>(q, nt, alone, sms, s);
    default: return launch_rows_hooks<3, 128>(q, nt, alone, sms, s);
  }
}

}  // namespace fltop
