// Beam extension, prefix merge, top-K selection and prefix-trie maintenance
// for frame-pruned CTC prefix beam search (Algorithm 1: the loops over the
// beam and over the surviving tokens, B'.add, SelectTopK, and
// GetHighestScorePrefix after the last frame).
//
// One thread block decodes one utterance and walks its frames serially; the
// beam lives in shared memory for the whole utterance.  The frame loop is a
// chain of dependent steps and nothing in it is bandwidth-bound: what bounds a
// frame is the longest chain of dependent instructions any one warp runs
// between two barriers.  The warps of a block therefore have roles:
//
//   stay warps   one lane per beam entry q: the "stay" candidate
//                (pb' = tot + lp[blank], pnb' = pnb + lp[last(q)]) and the
//                prefix merge.
//   ext warps    the (beam entry, non-blank survivor) extension candidates,
//                dealt out so that candidate e = q * S + j goes to ext lane
//                e mod NX; the extensions that end up selected come from the
//                few best entries, i.e. from consecutive e, and so land on
//                different lanes.
//   chore warp   everything a frame needs that is not on that chain: it
//                prefetches the survivor lists two frames ahead, clears the
//                next frame's tables, stages the next frame's log-probability
//                table and publishes its constants (survivor count, position
//                of blank, the reciprocal the ext lanes divide with).
//
// A frame:
//   P1  every candidate is evaluated once and counted in a histogram of its
//       score (1/4 nat per bin).  The prefix merge happens here: an entry
//       whose parent prefix is also in the beam (found through a small hash
//       table of the beam's prefix fingerprints) adds the mass of "parent
//       extended by last(q)" to its own pnb', takes that extension's count
//       out of the histogram again and flags it as merged.
//   B1
//   P2  the histogram is scanned for the bin that holds the K-th best score
//       (small blocks: every warp for itself, which saves a barrier).  The
//       upper edge of the first non-empty group of bins becomes the new zero
//       of the relative scores.
//   P3  candidates above the cut bin take consecutive beam slots from one
//       warp-aggregated counter and are written to the next beam, with their
//       fingerprint entered into the next frame's hash table and, for an
//       extension, a back-pointer node appended to the trie.  Candidates
//       inside the cut bin are listed and, after a barrier (B3), ranked
//       exactly among themselves (a handful).
//   B4
// If the cut bin is crowded (many near-equal scores) an exact radix select
// over order-preserving integer keys replaces the list.
//
// Prefix identity.  A prefix is its token sequence.  Each beam entry carries
// a 64-bit fingerprint of its sequence, fingerprint(child) =
// mix(fingerprint(parent), token), and the fingerprint of its parent.  Two
// candidates of a frame can name the same prefix only as "entry q stays" and
// "q's parent, also in the beam, extends by last(q)", so the merge needs the
// beam slot of q's parent and nothing else: a lookup of the parent's
// fingerprint among the beam's fingerprints.  This holds no matter how often
// a prefix has left and re-entered the beam, needs no per-prefix state in
// HBM, and keeps the trie append-only (8 bytes per entry that enters the
// beam).  Distinct sequences collide with probability 2^-64 per comparison.
//
// Scores are float32 relative to a per-frame reference within a few nats of
// the best total; the sum of the references is kept in float64.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "fltop_device.cuh"
#include "fltop_internal.h"

namespace fltop {
namespace {


__device__ __forceinline__ void cp_async8(void* smem_dst, const void* gmem_src) {
  const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(d), "l"(gmem_src));
}
__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gmem_src) {
  const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(d), "l"(gmem_src));
}
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(d), "l"(gmem_src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n"); }
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");
}
__device__ __forceinline__ void cp_async_wait_but_one() {
  asm volatile("cp.async.wait_group 1;\n" ::: "memory");
}

// Asynchronous bulk copy shared -> global (not multicast).  A block barrier does not wait for
// it, unlike an ordinary global store, whose acknowledgement the next barrier would sit out.
__device__ __forceinline__ void bulk_store(void* gmem_dst, const void* smem_src, unsigned bytes) {
  const unsigned s = (unsigned)__cvta_generic_to_shared(smem_src);
  asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;\n" ::"l"(gmem_dst),
               "r"(s), "r"(bytes)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;\n" ::: "memory");
}
// All but the most recent bulk copy have read their source.
__device__ __forceinline__ void bulk_store_wait_read_but_one() {
  asm volatile("cp.async.bulk.wait_group.read 1;\n" ::: "memory");
}
__device__ __forceinline__ void bulk_store_wait_all() {
  asm volatile("cp.async.bulk.wait_group 0;\n" ::: "memory");
}

// The fields of a beam entry that every candidate of the entry needs.
struct __align__(16) Hot {
  int last;    // last token of the prefix, -1 for the empty prefix
  float pb;    // log-mass of alignments ending in blank (relative)
  float pnb;   // ... ending in the last token
  float tot;   // lse(pb, pnb)
};
// Identity of a beam entry.
struct __align__(16) Ident {
  unsigned long long print;   // fingerprint of the token sequence
  unsigned long long pprint;  // fingerprint of the sequence without its last token
};
// Where a beam entry's tokens are: its trie node and its length.
struct __align__(8) Where {
  int node;
  int len;
};
// What a frame needs to know before it starts (written by the chore warp one frame ahead).
struct __align__(16) FrameInfo {
  int S;           // survivors of the frame
  int blank_j;     // position of blank among them, -1 if pruned
  int Snb;         // non-blank survivors
  float lp_blank;  // log-probability of blank, -inf if pruned
  float inv_s;     // 1 / max(Snb, 1)
  int dq, dj;      // (number of ext lanes) divmod max(Snb, 1)
  int pad;
};

enum {
  // one copy per frame parity
  SC_LISTN = 0, SC_SLOT, SC_SLOT_E, SC_MAXKEY, SC_WIN_E, SC_PER_FRAME,
  // single copies
  SC_THR = 2 * SC_PER_FRAME, SC_LEFT, SC_CUT_COUNT, SC_CUT_BASE, SC_TOTAL, SC_FIRST, SC_STATUS,
  SC_CREATED, SC_CLASHES, SC_EXACT, SC_DEAD, SC_NLIVE, SC_MADE, SC_MADE_ODD, SC_NEXT_S, SC_NEXT_BJ, SC_NEXT_BL, SC_KEPT,
  // exact fallback select
  SC_PREFIX, SC_SHIFT, SC_NEED, SC_TAKEALL, SC_DONE, SC_NBEAM_NEXT, SC_COUNT
};

// Slots of the beam's fingerprint table: a power of two, sixteen times the beam width for
// small beams (probe sequences of length one, almost always) and at least twice for large.
__host__ __device__ inline int table_size(int K) {
  const int want = K <= 128 ? 16 * K : (K <= 1024 ? 4 * K : 2 * K);
  int n = 256;
  while (n < want) n <<= 1;
  return n;
}
constexpr unsigned kEmptySlot = 0xffffffffu;  // table entry: [tag : 20][beam slot : 12]
// words of the bitmap over a frame's extension candidates (at most K * V of them)
__host__ __device__ inline int dup_words(int K, int V) { return (K * ((V + 31) / 32) + 3) & ~3; }
__host__ __device__ inline int node_stage_len(int K) { return (K + 1) & ~1; }

// Byte offsets of the shared-memory arrays.
// widest vocabulary whose frames the decode block prunes itself (one token per lane)
constexpr int kFusedMaxV = 32;
// ... and the widest whose frames it prunes itself with the chore warp walking the row
constexpr int kFusedWideMaxV = 1024;
__host__ __device__ inline int raw_row_len(int V) {
  return (V > kFusedMaxV && V <= kFusedWideMaxV) ? V : kFusedMaxV;
}
// up to this many stay lanes, every stay warp looks at all stay candidates itself (P3a)
constexpr int kOwnStayLanes = 128;

struct Lay {
  unsigned sv, hot, ident, where, nstage, finfo, warp_sums, st_pb, st_pnb, st_tot, dup, tab, lpv,
      jpos, hist,
      rhist, list_key, list_id, sel_key, sel_id, scal, raw, total;
};

__host__ __device__ inline Lay make_layout(int K, int V) {
  Lay l;
  unsigned off = 0;
  auto take = [&](unsigned bytes) {
    const unsigned at = off;
    off += (bytes + 15u) & ~15u;
    return at;
  };
  l.raw = take(4u * raw_row_len(V) * 4);  // first: its address needs no offset
  l.sv = take(4u * V * 8);
  l.hot = take(2u * K * 16);
  l.ident = take(2u * K * 16);
  l.where = take(2u * K * 8);
  l.nstage = take(2u * node_stage_len(K) * 8);
  l.finfo = take(2u * 32);
  l.warp_sums = take(34 * 8);
  l.st_pb = take(K * 4);
  l.st_pnb = take(K * 4);
  l.st_tot = take(K * 4);
  l.dup = take(2u * dup_words(K, V) * 4);
  l.tab = take(2u * table_size(K) * 4);
  l.lpv = take(2u * V * 4);
  l.jpos = take(2u * V * 4);
  l.hist = take(2u * kFastBins * 4);
  l.rhist = take(kPasses * kBins * 4);
  l.list_key = take(kListCap * 4);
  l.list_id = take(kListCap * 4);
  l.sel_key = take(K * 4);
  l.sel_id = take(K * 4);
  l.scal = take(SC_COUNT * 4);
  l.total = off;
  return l;
}

// Exclusive block scan of a packed pair of counters (low / high 32 bits).
__device__ __forceinline__ unsigned long long block_exclusive_scan(unsigned long long v,
                                                                   unsigned long long* warp_sums,
                                                                   unsigned long long* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_warps = (blockDim.x + 31) >> 5;
  unsigned long long inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long up = __shfl_up_sync(kFull, inc, o);
    if (lane >= o) inc += up;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    unsigned long long w = lane < n_warps ? warp_sums[lane] : 0ull;
    unsigned long long winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long up = __shfl_up_sync(kFull, winc, o);
      if (lane >= o) winc += up;
    }
    warp_sums[lane] = winc - w;  // exclusive prefix of each warp
    if (lane == 31) warp_sums[32] = winc;
  }
  __syncthreads();
  *total = warp_sums[32];
  return warp_sums[warp] + inc - v;
}

// Exact fallback select: after a histogram pass over one radix digit, warp 0
// finds the bin that holds the need-th largest key of the current prefix group.
__device__ __forceinline__ void resolve_digit(const unsigned* h, int* scal, int pass, int shift) {
  const int lane = threadIdx.x & 31;
  const int need = scal[SC_NEED];
  constexpr int PER = kBins / 32;  // lane l owns bins [255 - 8l - 7, 255 - 8l], walked from the top
  unsigned c = 0;
#pragma unroll
  for (int i = 0; i < PER; ++i) c += h[kBins - 1 - (lane * PER + i)];
  unsigned inc = c;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned up = __shfl_up_sync(kFull, inc, o);
    if (lane >= o) inc += up;
  }
  const unsigned total = __shfl_sync(kFull, inc, 31);
  if (pass == 0 && (int)total <= need) {
    if (lane == 0) {  // fewer candidates than beam slots: keep every candidate
      scal[SC_PREFIX] = 0; scal[SC_SHIFT] = 0; scal[SC_NEED] = 0; scal[SC_TAKEALL] = 0;
      scal[SC_DONE] = 1; scal[SC_NBEAM_NEXT] = (int)total;
    }
    return;
  }
  const unsigned hit = __ballot_sync(kFull, (int)inc >= need);
  const int owner = __ffs(hit) - 1;
  if (lane == owner) {
    unsigned acc = inc - c;
    int d = kBins - 1 - lane * PER;
    unsigned cnt = 0;
    for (int i = 0; i < PER; ++i, --d) {
      cnt = h[d];
      if ((int)(acc + cnt) >= need) break;
      acc += cnt;
    }
    const int left = need - (int)acc;
    scal[SC_PREFIX] = (int)(((unsigned)scal[SC_PREFIX] << kRadixBits) | (unsigned)d);
    scal[SC_SHIFT] = shift;
    scal[SC_NEED] = left;
    const int all = ((int)cnt == left);
    scal[SC_TAKEALL] = all;
    scal[SC_DONE] = (all || shift == 0) ? 1 : 0;
  }
}

// e divmod d for 0 <= e < 2^22 by a float reciprocal and one correction step.
__device__ __forceinline__ void divmod_small(int e, int d, float inv_d, int& q, int& r) {
  q = __float2int_rz(((float)e + 0.5f) * inv_d);
  r = e - q * d;
  if (r < 0) { --q; r += d; }
  else if (r >= d) { ++q; r -= d; }
}

// KMAX / VMAX > 0: the shared-memory arrays are laid out for that beam width and vocabulary
// whatever K and V are (K <= KMAX, V <= VMAX), so every array offset is a compile-time
// constant; 0: laid out for the K and V of the call; -1: likewise, for wide beams (a crowded
// cut bin is split a second time, and the warps are shared out between the two kinds of
// candidate anew every frame).
// BT: an option of Algorithm 1 beyond N and R is on - beam_threshold (the exact best score of
// every frame is tracked) and / or merging by max instead of log-sum.
// CLK: every warp of block 0 records the SM clock at its phase boundaries (profiling; only the
// instantiations for blocks of up to 1024 threads without options exist with it).
template <int MAXT, int KMAX, int VMAX, bool BT, bool CLK = false>
__global__ void __launch_bounds__(MAXT) decode_kernel(DecodeParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int tid = threadIdx.x, NT = blockDim.x, lane = tid & 31;
  const int b = p.first_wave > 0 ? utterance_by_length(p.lengths, p.B, p.T, p.first_wave,
                                                        reinterpret_cast<int*>(smem))
                                 : (int)blockIdx.x;
  const int K = p.K, V = p.V, blank = p.blank;
  const int KS = KMAX > 0 ? KMAX : K;  // strides of the per-entry / per-token arrays
  constexpr bool kWide = KMAX < 0;
  constexpr int kBitsOfK = KMAX == 64 ? 7 : 12;  // bits of the widest beam (the histogram scan counts over them)
  // rows of more than 32 tokens pruned inside: compiled only into the instantiations that can
  // meet them (their code costs the character-vocabulary ones a few per cent even when idle)
  constexpr bool kWideRows = VMAX != 32;
  const int VS = VMAX > 0 ? VMAX : V;
  const Lay L = make_layout(KS, VS);
  // (a caller may shrink the table: only the test of the bounded probe walks does)
  const int TS = p.table_slots > 0 ? min(p.table_slots, table_size(KS)) : table_size(KS);
  const int DW = dup_words(KS, VS);
  const int NSL = node_stage_len(KS);
  const unsigned tmask = (unsigned)TS - 1u;
  const unsigned lt_mask = (1u << lane) - 1u;

  Survivor* const sv_base = reinterpret_cast<Survivor*>(smem + L.sv);
  Hot* const hot_base = reinterpret_cast<Hot*>(smem + L.hot);
  Ident* const ident_base = reinterpret_cast<Ident*>(smem + L.ident);
  Where* const where_base = reinterpret_cast<Where*>(smem + L.where);
  FrameInfo* const finfo = reinterpret_cast<FrameInfo*>(smem + L.finfo);
  unsigned long long* const warp_sums = reinterpret_cast<unsigned long long*>(smem + L.warp_sums);
  float* const st_pb = reinterpret_cast<float*>(smem + L.st_pb);
  float* const st_pnb = reinterpret_cast<float*>(smem + L.st_pnb);
  float* const st_tot = reinterpret_cast<float*>(smem + L.st_tot);  // lse(st_pb, st_pnb)
  unsigned* const dup_base = reinterpret_cast<unsigned*>(smem + L.dup);
  TrieNode* const nstage = reinterpret_cast<TrieNode*>(smem + L.nstage);
  int* const jpos_base = reinterpret_cast<int*>(smem + L.jpos);
  unsigned* const tab_base = reinterpret_cast<unsigned*>(smem + L.tab);
  float* const lpv_base = reinterpret_cast<float*>(smem + L.lpv);
  unsigned* const hist_base = reinterpret_cast<unsigned*>(smem + L.hist);
  unsigned* const rhist = reinterpret_cast<unsigned*>(smem + L.rhist);
  unsigned* const list_key = reinterpret_cast<unsigned*>(smem + L.list_key);
  int* const list_id = reinterpret_cast<int*>(smem + L.list_id);
  unsigned* const sel_key = reinterpret_cast<unsigned*>(smem + L.sel_key);
  int* const sel_id = reinterpret_cast<int*>(smem + L.sel_id);
  int* const scal = reinterpret_cast<int*>(smem + L.scal);

  // ---- roles -----------------------------------------------------------------------
  const int NW = NT >> 5, warp = tid >> 5;
  int nsw = (K + 31) >> 5;                   // stay warps: one lane per beam entry if possible
  if (nsw > (NW - 1) / 2) nsw = (NW - 1) / 2;
  if (nsw < 1) nsw = 1;
  // (wide beams move this split every frame, see the frame loop)
  int NS = nsw << 5;                         // stay lanes
  int NX = (NW - 1 - nsw) << 5;              // ext lanes
  const bool is_chore = warp == NW - 1;
  bool is_stay = warp < nsw;
  bool is_ext = !is_chore && !is_stay;
  int xl = tid - NS;                         // index among the ext lanes
  const bool warp_scans = NT <= kSmallBlock;
  // the options live in instantiations of their own (BT): the default one has neither
  const bool use_bt = BT && p.beam_threshold > 0.f;
  const bool use_max = BT && p.merge_max != 0;

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
  TrieNode* nodes = p.nodes + (int64_t)b * p.nodes_per_utt;
  int32_t* st = p.streaming
                    ? p.state + (int64_t)b * (kStateHeaderWords + kStateWordsPerSlot * (int64_t)K)
                    : nullptr;

  // ---- initialise shared state -------------------------------------------------
  for (int i = tid; i < 2 * DW; i += NT) dup_base[i] = 0u;
  for (int i = tid; i < 2 * TS; i += NT) tab_base[i] = kEmptySlot;
  for (int i = tid; i < 2 * VS; i += NT) lpv_base[i] = neg_inf();
  for (int i = tid; i < 2 * kFastBins; i += NT) hist_base[i] = 0u;
  if (tid < SC_COUNT) scal[tid] = tid == SC_NEXT_BJ ? -1 : 0;
  int created = 0, live_sum = 0, tag_clashes = 0;
  int cur = 0, nb, n_nodes, frames_seen;
  double offset;
  if (do_reset) {
    nb = bad_len && !p.streaming ? 0 : 1;
    n_nodes = 2;  // node 0 is the empty prefix, id 1 is not used: blocks of ids start even
    offset = 0.0;
    frames_seen = 0;
    if (tid == 0) {
      Hot e;
      e.last = -1; e.pb = 0.f; e.pnb = neg_inf(); e.tot = 0.f;
      hot_base[0] = e;
      ident_base[0] = Ident{kRootPrint, 0ull};
      where_base[0] = Where{0, 0};
      nodes[0] = TrieNode{-1, -1};
    }
  } else {
    const StateHeader* hd = reinterpret_cast<const StateHeader*>(st);
    nb = hd->nbeam; n_nodes = hd->n_nodes; frames_seen = hd->frames; offset = hd->offset;
    status |= hd->status;
    const int32_t* a = st + kStateHeaderWords;
    for (int i = tid; i < nb; i += NT) {
      Hot e;
      e.last = a[K + i];
      e.pb = __int_as_float(a[3 * K + i]);
      e.pnb = __int_as_float(a[4 * K + i]);
      e.tot = __int_as_float(a[5 * K + i]);
      hot_base[i] = e;
      where_base[i] = Where{a[i], a[2 * K + i]};
      ident_base[i] = Ident{reinterpret_cast<const unsigned long long*>(a + 6 * K)[i],
                            reinterpret_cast<const unsigned long long*>(a + 8 * K)[i]};
    }
  }
  __syncthreads();

  // Hash table of the beam's fingerprints.  An entry holds a beam slot and 20 bits of its
  // fingerprint, so a probe that meets another prefix is rejected without a second load; a
  // tag match is confirmed against the full fingerprint.  The table is at most half full, so a
  // probe sequence ends at an empty entry long before it has gone round; should it ever go
  // round (back at its first slot), the walk gives up and the utterance is flagged FLTOP_ST_INTERNAL.
  auto table_insert = [&](unsigned* tab, unsigned long long h, int slot) {
    const unsigned val = (((unsigned)h & 0xfffffu) << 12) | (unsigned)slot;
    const unsigned home = (unsigned)(h >> 40) & tmask;
    unsigned pos = home;
    do {
      if (atomicCAS(&tab[pos], kEmptySlot, val) == kEmptySlot) return;
      pos = (pos + 1) & tmask;
    } while (pos != home);
    atomicOr(&scal[SC_STATUS], 16);  // FLTOP_ST_INTERNAL: the entry is not in the table
  };
  // Beam slot of the entry with fingerprint h, or -1.
  auto table_find = [&](const unsigned* tab, const Ident* ids, unsigned long long h) {
    const unsigned tag = (unsigned)h & 0xfffffu;
    const unsigned home = (unsigned)(h >> 40) & tmask;
    unsigned pos = home;
    do {
      const unsigned v = tab[pos];
      if (v == kEmptySlot) return -1;
      if ((v >> 12) == tag) {
        const int slot = (int)(v & 0xfffu);
        if (ids[slot].print == h) return slot;
        ++tag_clashes;  // same 20-bit tag, another sequence
      }
      pos = (pos + 1) & tmask;
    } while (pos != home);
    atomicOr(&scal[SC_STATUS], 16);  // FLTOP_ST_INTERNAL
    return -1;
  };

  const int32_t* counts = p.counts + (int64_t)b * p.T;
  const Survivor* entries = p.entries + (int64_t)b * p.T * V;
  auto svbuf = [&](int t) -> Survivor* { return sv_base + (t & 3) * VS; };
  auto lpvbuf = [&](int t) -> float* { return lpv_base + (t & 1) * VS; };

  // The tables of frame t1 (its survivors are in shared memory): token -> log-probability and
  // token -> position in the survivor list; the table of frame t1 - 1 is forgotten (t1 > 0).
  // Threads first, first + stride, ... share the work; whoever meets blank notes where.
  auto stage_tables = [&](int t1, int S_prev, int S1, int first, int stride) {
    if (t1 > 0) {
      float* lp_old = lpvbuf(t1 - 1);
      const Survivor* so = svbuf(t1 - 1);
      for (int j = first; j < S_prev; j += stride) lp_old[so[j].token] = neg_inf();
    }
    float* lp_new = lpvbuf(t1);
    int* jp_new = jpos_base + (t1 & 1) * VS;
    const Survivor* sn = svbuf(t1);
    for (int j = first; j < S1; j += stride) {
      const Survivor s = sn[j];
      lp_new[s.token] = s.logp;
      jp_new[s.token] = j;
      if (s.token == blank) {
        scal[SC_NEXT_BJ] = j;
        scal[SC_NEXT_BL] = __float_as_int(s.logp);
      }
    }
  };
  // One thread, once the tables of frame t1 are complete: the constants of the frame.
  auto publish_frame = [&](int t1, int S1) {
    FrameInfo f;
    f.S = S1;
    f.blank_j = scal[SC_NEXT_BJ];
    f.lp_blank = f.blank_j >= 0 ? __int_as_float(scal[SC_NEXT_BL]) : neg_inf();
    f.Snb = S1 - (f.blank_j >= 0 ? 1 : 0);
    const int d = max(f.Snb, 1);
    f.inv_s = 1.f / (float)d;
    divmod_small(NX, d, f.inv_s, f.dq, f.dj);
    f.pad = 0;
    finfo[t1 & 1] = f;
    scal[SC_NEXT_BJ] = -1;
  };

  // Fused pruning (V <= 32, emissions given): the chore warp fetches the raw rows itself, three
  // frames ahead, and applies the relative threshold (Algorithm 1's conditional break) and
  // the top-N cap of stage 1 in registers, one token per lane; no survivor list ever goes
  // through HBM.  The survivor list it leaves in shared memory is the prune kernel's: tokens
  // in ascending order, a tie at the N-th place goes to the lower token id.
  // (Nothing of this is kept in registers across the frame loop: the large blocks have 64 a
  // thread, and every thread would pay for what only the chore warp uses.)
  auto fused = [&]() -> bool { return p.logp != nullptr; };
  const int RS = raw_row_len(VS);  // floats between the raw rows of consecutive frames
  auto raw_row = [&](int t1) -> float* {
    return reinterpret_cast<float*>(smem) + (t1 & 3) * RS;
  };
  // float32 rows: a word per lane; fp16 / bf16 rows: a word holds two tokens (V is even then)
  auto fetch_row = [&](int t1) {
    const int64_t at = (int64_t)b * p.stride_b + (int64_t)t1 * p.stride_t;
    if (kWideRows && V > kFusedMaxV) {
      // a wide row (float32, 16-byte aligned, V a multiple of four): 16 bytes per lane and turn
      const float* src = static_cast<const float*>(p.logp) + at;
      for (int c = 4 * lane; c < V; c += 128) cp_async16(raw_row(t1) + c, src + c);
    } else if (p.dtype == kEmissionF32) {
      if (lane < V) cp_async4(raw_row(t1) + lane, static_cast<const float*>(p.logp) + at + lane);
    } else if (2 * lane < V) {
      cp_async4(raw_row(t1) + lane, static_cast<const uint16_t*>(p.logp) + at + 2 * lane);
    }
  };
  // the row of frame t1 has landed; returns the survivor count
  // order-preserving integer key of a float32 (a NaN sorts below every number)
  auto okey = [](float v) -> unsigned {
    const unsigned vu = __float_as_uint(v);
    return (v == v) ? ((vu & 0x80000000u) ? ~vu : (vu | 0x80000000u)) : 0x007fffffu;
  };
  // A row of more than 32 tokens (V a multiple of four): the chore warp walks it twice, four
  // tokens per lane and turn - first the row maximum and with it the threshold, then the
  // survivors in ascending token order.  The two walks are separate calls: within the frame
  // loop each takes a stretch in which the chore warp would otherwise wait.
  auto wide_row_threshold = [&](int t1) -> float {
    const float4* const row = reinterpret_cast<const float4*>(raw_row(t1));
    float m = neg_inf();
    for (int c = lane; 4 * c < V; c += 32) {
      const float4 x = row[c];
      m = fmaxf(m, fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w)));  // (a NaN never is the maximum)
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, o));
    return __fadd_rn(m, p.log_r);
  };
  // (tokens [4 * from, 4 * to) of the row, appended to the n survivors found so far)
  auto wide_row_survivors = [&](int t1, float thr, int from, int to, int n) -> int {
    const float4* const row = reinterpret_cast<const float4*>(raw_row(t1));
    Survivor* const out = svbuf(t1);
    for (int c0 = from; c0 < to; c0 += 32) {
      const int c = c0 + lane;
      const bool in = c < to;
      const float4 x = in ? row[c] : make_float4(0.f, 0.f, 0.f, 0.f);
      const bool k0 = in && x.x >= thr, k1 = in && x.y >= thr, k2 = in && x.z >= thr,
                 k3 = in && x.w >= thr;
      const unsigned b0 = __ballot_sync(kFull, k0), b1 = __ballot_sync(kFull, k1),
                     b2 = __ballot_sync(kFull, k2), b3 = __ballot_sync(kFull, k3);
      // tokens 4c .. 4c+3 of lane c come after everything the lanes before it keep
      int at = n + __popc(b0 & lt_mask) + __popc(b1 & lt_mask) + __popc(b2 & lt_mask) +
               __popc(b3 & lt_mask);
      if (k0) out[at++] = Survivor{4 * c, x.x};
      if (k1) out[at++] = Survivor{4 * c + 1, x.y};
      if (k2) out[at++] = Survivor{4 * c + 2, x.z};
      if (k3) out[at++] = Survivor{4 * c + 3, x.w};
      n += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
    }
    return n;
  };
  const int wide_half = ((V / 4 + 63) / 64) * 32;  // float4s of the first half of a wide row
  auto prune_wide_row = [&](int t1) -> int {
    const int n = wide_row_survivors(t1, wide_row_threshold(t1), 0, V / 4, 0);
    if (lane == 0) scal[SC_KEPT] += n;
    return n;
  };
  auto prune_row = [&](int t1) -> int {
    if (kWideRows && V > kFusedMaxV) return prune_wide_row(t1);
    float v = neg_inf();
    if (p.dtype == kEmissionF32) {
      if (lane < V) v = raw_row(t1)[lane];  // the word this lane fetched itself
    } else {
      __syncwarp();  // the word was fetched by lane / 2
      if (lane < V) {
        const unsigned short bits = reinterpret_cast<const unsigned short*>(raw_row(t1))[lane];
        v = p.dtype == kEmissionF16 ? __half2float(__ushort_as_half(bits))
                                    : __bfloat162float(__ushort_as_bfloat16(bits));
      }
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
      // order-preserving integer key; 0 = not (or no longer) in the running
      const unsigned u = __float_as_uint(v);
      unsigned key = keep ? ((u & 0x80000000u) ? ~u : (u | 0x80000000u)) : 0u;
      unsigned chosen = 0u;
      for (int i = 0; i < p.top_n; ++i) {
        const unsigned best_key = __reduce_max_sync(kFull, key);
        const int w = __ffs(__ballot_sync(kFull, key == best_key)) - 1;
        chosen |= 1u << w;
        if (lane == w) key = 0u;
      }
      kept = chosen;
    }
    if ((kept >> lane) & 1u) svbuf(t1)[__popc(kept & lt_mask)] = Survivor{lane, v};
    const int n = __popc(kept);
    if (lane == 0) {
      scal[SC_KEPT] += n;  // survivors over all frames of this call
      if (p.dbg_masks) p.dbg_masks[(int64_t)b * p.T + t1] = kept;  // instrumented launches only
    }
    return n;
  };

  // ---- prologue: survivors of frames 0 and 1, tables of frame 0 ----------------------
  int c0 = 0, c1 = 0, c2 = 0;  // survivor counts of frames t, t+1, t+2 (chore warp only)
  for (int i = tid; i < nb; i += NT) table_insert(tab_base, ident_base[i].print, i);
  if (is_chore && fused()) {
    if (len > 0) fetch_row(0);
    if (len > 1) fetch_row(1);
    cp_async_commit();
    if (len > 2) fetch_row(2);
    cp_async_commit();
    cp_async_wait_but_one();
    c0 = len > 0 ? prune_row(0) : 0;
    c1 = len > 1 ? prune_row(1) : 0;
    __syncwarp();
  } else if (is_chore) {
    c0 = len > 0 ? counts[0] : 0;
    c1 = len > 1 ? counts[1] : 0;
    c2 = len > 2 ? counts[2] : 0;
    for (int j = lane; j < c0; j += 32) cp_async8(&svbuf(0)[j], &entries[j]);
    cp_async_commit();
    for (int j = lane; j < c1; j += 32) cp_async8(&svbuf(1)[j], &entries[(int64_t)V + j]);
    cp_async_commit();
    cp_async_wait_all();
    __syncwarp();
  }
  if (is_chore) {
    stage_tables(0, 0, c0, lane, 32);
    __syncwarp();
    if (lane == 0) publish_frame(0, c0);
  }
  __syncthreads();

  int pend_at = 0;
  unsigned pend_bytes = 0u;
  for (int t = 0; t < len; ++t) {
    const int par = t & 1, nxt = cur ^ 1;
    // marks: 0 frame start, 1 candidates evaluated, 2 past B1, 3 the cut is known, 4 candidates
    // settled (before B3), 5 at B2 (large blocks), 6 next beam written (before B4), 7 past B4
    auto clock_mark = [&](int i) {
      if (CLK && blockIdx.x == 0 && lane == 0 && p.dbg_clocks && t >= p.dbg_frame0 &&
          t < p.dbg_frame0 + p.dbg_frames)
        p.dbg_clocks[((int64_t)(t - p.dbg_frame0) * 32 + warp) * 8 + i] = clock64();
    };
    clock_mark(0);
    const Survivor* const sv = svbuf(t);
    const float* const lpv = lpvbuf(t);
    const Hot* const hc = hot_base + cur * KS;
    Hot* const hn = hot_base + nxt * KS;
    const Ident* const id_c = ident_base + cur * KS;
    Ident* const id_n = ident_base + nxt * KS;
    const Where* const wh_c = where_base + cur * KS;
    Where* const wh_n = where_base + nxt * KS;
    unsigned* const hist = hist_base + par * kFastBins;
    unsigned* const dupbits = dup_base + par * DW;
    const int* const jpos = jpos_base + par * VS;
    const unsigned* const tab_c = tab_base + par * TS;
    unsigned* const tab_n = tab_base + (par ^ 1) * TS;
    int* const sc_c = scal + par * SC_PER_FRAME;

    const FrameInfo fi = finfo[par];
    const int Snb = fi.Snb, blank_j = fi.blank_j;
    const int Sdiv = max(Snb, 1);
    const int next = nb * Snb;  // extension candidates of this frame
    int dq = fi.dq, dj = fi.dj;  // (q, j) step between a lane's successive extension candidates
    if (kWide) {
      // Wide beams share the warps out anew every frame, by the counts of the two kinds of
      // candidate; a stay candidate takes about as long as four extension candidates.
      const int ws = 4 * nb, wx = next;
      int n = ((NW - 1) * ws + ws + wx - 1) / (ws + wx);
      n = max(1, min(n, min((nb + 31) >> 5, NW - 2)));
      NS = n << 5;
      NX = (NW - 1 - n) << 5;
      is_stay = warp < n;
      is_ext = !is_chore && !is_stay;
      xl = tid - NS;
      divmod_small(NX, Sdiv, fi.inv_s, dq, dj);
    }

    // position of the j-th non-blank survivor in the survivor list
    const int blank_at = blank_j >= 0 ? blank_j : 0x7fffffff;
    auto sv_index = [&](int j) -> int { return j + (j >= blank_at ? 1 : 0); };
    // score of entry e extended by non-blank survivor j
    auto ext_score = [&](const Hot& e, int j) -> float {
      const Survivor s = sv[sv_index(j)];
      return ((s.token == e.last) ? e.pb : e.tot) + s.logp;
    };
    auto ext_key = [&](const Hot& e, int j) -> unsigned { return score_key(ext_score(e, j)); };
    auto ext_token = [&](int j) -> int { return sv[sv_index(j)].token; };
    // extension candidate e = q * Snb + j names a prefix that is already in the beam
    auto merged = [&](int e) -> bool { return (dupbits[e >> 5] >> (e & 31)) & 1u; };
    auto count = [&](float score) { atomicAdd(&hist[score_bin(score)], 1u); };
    // stay candidate of entry q, including the prefix merge
    auto stay_eval = [&](int q) -> float {
      const Hot e = hc[q];
      const float npb = e.tot + fi.lp_blank;
      float own = neg_inf(), dup = neg_inf();  // non-blank mass: the entry's own, its parent's
      if (e.last >= 0) {
        const float le = lpv[e.last];
        own = e.pnb + le;
        const int pq = table_find(tab_c, id_c, id_c[q].pprint);
        if (pq >= 0) {
          const Hot pe = hc[pq];
          dup = ((pe.last == e.last) ? pe.pb : pe.tot) + le;
          if (dup != neg_inf()) {  // the parent's extension by last(q) names this prefix
            atomicSub(&hist[score_bin(dup)], 1u);
            const int jp = jpos[e.last];  // position among all survivors -> among non-blank
            const int ed = pq * Snb + jp - ((blank_j >= 0 && jp > blank_j) ? 1 : 0);
            atomicOr(&dupbits[ed >> 5], 1u << (ed & 31));
          }
        }
      }
      // masses are summed, or (merge_max) the better one is taken.  The total is formed from
      // the three terms directly, not from npnb: the two results do not wait for each other.
      const float npnb = use_max ? fmaxf(own, dup) : lse2(own, dup);
      const float tot = use_max ? fmaxf(npb, fmaxf(own, dup)) : lse3(npb, own, dup);
      st_pb[q] = npb;
      st_pnb[q] = npnb;
      st_tot[q] = tot;
      if (tot != neg_inf()) count(tot);
      return tot;
    };
    // this lane's extension candidates: e_first, e_first + NX, ... as (q, j) pairs
    int q0 = 0, j0 = 0;
    auto step = [&](int& q, int& j) {
      q += dq;
      j += dj;
      if (j >= Sdiv) { j -= Sdiv; ++q; }
    };
    // (q, j) of this lane's k-th extension candidate
    auto nth = [&](int k, int& q, int& j) {
      q = q0 + k * dq;
      j = j0 + k * dj;
      while (j >= Sdiv) { j -= Sdiv; ++q; }
    };

    // Chore warp: the nodes staged by frame t-1 go to the trie; the histogram, the merge
    // bitmap, the counters (and, in small blocks, the hash table) of frame t+1 start empty.
    // Narrow beams do this after B1, where the scan leaves the chore warp time to spare; with
    // wide beams the first phase is the long one, so it goes there.
    auto chore_window = [&]() {
      if (lane == 0 && pend_bytes) {
        bulk_store(nodes + pend_at, nstage + (par ^ 1) * NSL, pend_bytes);
        bulk_store_wait_read_but_one();  // the staging buffer of this frame is free again
      }
      const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
      const uint4 ones = make_uint4(~0u, ~0u, ~0u, ~0u);
      uint4* hist_n = reinterpret_cast<uint4*>(hist_base + (par ^ 1) * kFastBins);
      uint4* dup_n = reinterpret_cast<uint4*>(dup_base + (par ^ 1) * DW);
      uint4* tb_n = reinterpret_cast<uint4*>(tab_n);
      for (int i = lane; i < kFastBins / 4; i += 32) hist_n[i] = zero;
      for (int i = lane; i < DW / 4; i += 32) dup_n[i] = zero;
      if (warp_scans)  // (large blocks share this out among all warps)
        for (int i = lane; i < TS / 4; i += 32) tb_n[i] = ones;
      if (lane < SC_PER_FRAME) scal[(par ^ 1) * SC_PER_FRAME + lane] = 0;
    };
    // ---- P1: every candidate is evaluated once and counted -----------------------------
    float wide_thr = neg_inf();  // (chore warp, wide rows) the threshold of frame t+2 ...
    int wide_n = 0;              // ... and the survivors of its first half
    float kc[kCache];  // this ext lane's first extension scores (-inf: none)
#pragma unroll
    for (int k = 0; k < kCache; ++k) kc[k] = neg_inf();
    float my_max = neg_inf();  // best score among this thread's candidates (beam_threshold only)
    if (is_stay) {
      for (int i = tid; i < nb; i += NS) {
        const float sc = stay_eval(i);
        if (use_bt) my_max = fmaxf(my_max, sc);
      }
    } else if (is_ext) {
      divmod_small(xl, Sdiv, fi.inv_s, q0, j0);
      int q = q0, j = j0;
#pragma unroll
      for (int k = 0; k < kCache; ++k) {
        if (xl + k * NX < next) {
          const float sc = ext_score(hc[q], j);
          step(q, j);
          kc[k] = sc;
          if (use_bt) my_max = fmaxf(my_max, sc);
          if (sc != neg_inf()) count(sc);
        }
      }
      for (int e = xl + kCache * NX; e < next; e += NX) {
        const float sc = ext_score(hc[q], j);
        step(q, j);
        if (use_bt) my_max = fmaxf(my_max, sc);
        if (sc != neg_inf()) count(sc);
      }
    } else {
      // chore warp: the emissions of frame t+3 (fused pruning) or the survivors of frame t+2
      // start their way to shared memory, and the row of frame t+2 becomes its survivor list;
      // the rest of its work waits until after B1, where nobody is waiting for it
      if (fused()) {
        if (t + 3 < len) fetch_row(t + 3);
      } else if (t + 2 < len) {
        const Survivor* src = entries + (int64_t)(t + 2) * V;
        Survivor* dst = svbuf(t + 2);
        for (int j = lane; j < c2; j += 32) cp_async8(&dst[j], &src[j]);
      }
      cp_async_commit();
      if (kWide) {
        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
        for (int i = lane; i < kFastBins / 4; i += 32) reinterpret_cast<uint4*>(rhist)[i] = zero;
      }
      if (lane == 0) scal[SC_NEXT_S] = c1;
      cp_async_wait_but_one();  // what was requested a frame ago has landed (visible after B1)
      if (fused()) {
        if (!kWideRows || V <= kFusedMaxV) c2 = (t + 2 < len) ? prune_row(t + 2) : 0;
        else if (t + 2 < len) {
          // a wide row: the threshold and the survivors of its first half now, the rest in P3
          wide_thr = wide_row_threshold(t + 2);
          wide_n = wide_row_survivors(t + 2, wide_thr, 0, min(wide_half, V / 4), 0);
        }
      }
      if (kWide) chore_window();
    }
    if (use_bt && !is_chore) {
      // SelectTopK's beam_threshold is relative to the exact best score of the frame
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) my_max = fmaxf(my_max, __shfl_xor_sync(kFull, my_max, o));
      if (lane == 0 && my_max != neg_inf())
        atomicMax(reinterpret_cast<unsigned*>(&sc_c[SC_MAXKEY]), score_key(my_max));
    }
    clock_mark(1);
    __syncthreads();  // B1
    clock_mark(2);

    // (chore warp, wide rows) the second half of frame t+2's survivors; returns their number
    auto finish_wide_row = [&]() -> int {
      if (t + 2 >= len) return 0;
      const int n = wide_row_survivors(t + 2, wide_thr, min(wide_half, V / 4), V / 4, wide_n);
      if (lane == 0) scal[SC_KEPT] += n;
      return n;
    };
    // ---- P2: the cut -------------------------------------------------------------------
    // The chore warp does not scan: while the others do, it stages the log-prob table and
    // the constants of frame t+1 (and fetches the survivor count of frame t+3); it takes
    // the cut from warp 0.
    auto chore_between = [&]() {
      const int c3 = (!fused() && t + 3 < len) ? counts[t + 3] : 0;
      if (t + 1 < len) {
        stage_tables(t + 1, c0, c1, lane, 32);
        __syncwarp();
        if (lane == 0) publish_frame(t + 1, c1);
      }
      if (!kWide) chore_window();
      c0 = c1; c1 = c2; c2 = c3;
    };
    auto publish_cut = [&](const Cut& c) {
      scal[SC_THR] = c.thr; scal[SC_LEFT] = c.left; scal[SC_CUT_COUNT] = c.cut_count;
      scal[SC_CUT_BASE] = c.cut_base; scal[SC_TOTAL] = c.total; scal[SC_FIRST] = c.first;
    };
    auto read_cut = [&](Cut& c) {
      c.thr = scal[SC_THR]; c.left = scal[SC_LEFT]; c.cut_count = scal[SC_CUT_COUNT];
      c.cut_base = scal[SC_CUT_BASE]; c.total = scal[SC_TOTAL]; c.first = scal[SC_FIRST];
    };
    Cut cut;
    if (warp_scans) {
      if (!is_chore) {
        cut = scan_score_histogram_ballots<kBitsOfK>(hist, K);
        if (warp == 0) {
          if (lane == 0) publish_cut(cut);
          __threadfence_block();
          asm volatile("bar.arrive 1, 64;" ::: "memory");  // releases the chore warp
        }
      } else {
        chore_between();
        asm volatile("bar.sync 1, 64;" ::: "memory");      // warp 0 has published the cut
        read_cut(cut);
      }
    } else {
      // large blocks: warp 0 scans, all the others stage the tables of frame t+1 together
      const int S_next = scal[SC_NEXT_S];
      if (warp == 0) {
        cut = scan_score_histogram_ballots<kBitsOfK>(hist, K);
        if (lane == 0) publish_cut(cut);
      } else {
        if (t + 1 < len) stage_tables(t + 1, fi.S, S_next, tid - 32, NT - 32);
        // the hash table of the next beam starts empty (first insertions come after B3)
        const uint4 ones = make_uint4(~0u, ~0u, ~0u, ~0u);
        uint4* tb_n = reinterpret_cast<uint4*>(tab_n);
        for (int i = tid - 32; i < TS / 4; i += NT - 32) tb_n[i] = ones;
        if (!kWide && is_chore) chore_window();
      }
      clock_mark(5);
      __syncthreads();  // B2 (large blocks only)
      read_cut(cut);
      if (is_chore) {
        const int c3 = (!fused() && t + 3 < len) ? counts[t + 3] : 0;
        if (lane == 0 && t + 1 < len) publish_frame(t + 1, S_next);
        c0 = c1; c1 = c2; c2 = c3;
      }
    }
    clock_mark(3);
    // new zero of the relative scores: the upper edge of the first non-empty group of bins
    const float best = -(float)(cut.first * kBinsPerLane) * (1.f / kBinsPerNat);
    const bool take_all = cut.cut_count == cut.left;  // also true when there is no cut at all
    const bool use_list = !take_all && cut.cut_count <= kListCap;
    int nbn = min(cut.total, K);
    // beam_threshold: a selected candidate scoring below (best of the frame) - threshold is
    // dropped.  Its beam slot is written as a dead entry (probability 0, no identity).
    float f_floor = neg_inf();
    if (use_bt) {
      const unsigned mk = (unsigned)sc_c[SC_MAXKEY];
      if (mk) f_floor = key_score(mk) - p.beam_threshold;
    }
    auto place_dead = [&](int slot) {
      Hot e;
      e.last = -1; e.pb = e.pnb = e.tot = neg_inf();
      hn[slot] = e;
      id_n[slot] = Ident{0ull, 0ull};
      wh_n[slot] = Where{0, 0};
      atomicAdd(&scal[SC_DEAD], 1);
    };
    TrieNode* const nst = nstage + par * NSL;
    // the frame's new prefixes get the node ids n_nodes, n_nodes + 1, ...
    const bool arena_ok = (int64_t)n_nodes + ((K + 1) & ~1) <= p.nodes_per_utt;

    // ---- P3: selected candidates take their slots in the next beam ---------------------
    auto place_stay = [&](int q, unsigned key, int slot) {
      if ((unsigned)slot >= (unsigned)K) return;  // only reachable with NaN scores
      if (use_bt && key_score(key) < f_floor) return place_dead(slot);
      Hot e;
      e.last = hc[q].last;
      e.pb = st_pb[q] - best;
      e.pnb = st_pnb[q] - best;
      e.tot = key_score(key) - best;
      hn[slot] = e;
      const Ident id = id_c[q];
      id_n[slot] = id;
      wh_n[slot] = wh_c[q];
      table_insert(tab_n, id.print, slot);
    };
    // a new prefix; `ord` numbers the frame's new prefixes (its trie record and node id)
    auto place_ext = [&](int q, int tok, unsigned key, int slot, int ord) {
      if ((unsigned)slot >= (unsigned)K || (unsigned)ord >= (unsigned)K) return;
      if (use_bt && key_score(key) < f_floor) return place_dead(slot);
      const float sc = key_score(key) - best;
      Hot e;
      e.last = tok; e.pb = neg_inf(); e.pnb = sc; e.tot = sc;
      hn[slot] = e;
      const unsigned long long hp = id_c[q].print;
      const unsigned long long h = child_print(hp, tok);
      id_n[slot] = Ident{h, hp};
      table_insert(tab_n, h, slot);
      const Where w = wh_c[q];
      // back-pointer node: staged here, written to the trie in one piece after the frame
      nst[ord] = TrieNode{w.node, tok};
      ++created;
      wh_n[slot] = Where{arena_ok ? n_nodes + ord : 0, w.len + 1};
    };
    // a candidate by its id: beam entry in the high half, 0 (stay) or j + 1 (extension by the
    // j-th non-blank survivor) in the low half
    auto place_by_id = [&](int id, unsigned key, int slot, int ord) {
      const int q = id >> 16, j1 = id & 0xffff;
      if (j1 == 0) place_stay(q, key, slot);
      else place_ext(q, ext_token(j1 - 1), key, slot, ord);
    };

    // the cut as scores (bin edges): score > f_hi is above the cut bin, score > f_lo is in it
    // or above.  A score of -inf passes neither.
    const float hi_edge = -(float)cut.thr * (1.f / kBinsPerNat);
    const float f_lo = (cut.thr >= kFastBins - 1) ? neg_inf()
                                                  : -(float)(cut.thr + 1) * (1.f / kBinsPerNat);
    const float f_hi = take_all ? f_lo : (cut.thr == 0 ? __int_as_float(0x7f800000) : hi_edge);
    // A crowded cut bin (wide beams) is split once more, into 256 sub-bins over its quarter
    // nat, and the cut is located among those.
    auto sub_bin = [&](float sc) -> int {
      const int b2 = __float2int_rz((hi_edge - sc) * (kBinsPerNat * (float)kFastBins));
      return min(kFastBins - 1, max(0, b2));
    };
    bool refined = false;
    int sub_thr = 0, sub_left = 0, sub_count = 0;
    if (kWide && !take_all && !use_list && cut.thr < kFastBins - 1) {
      unsigned* const h2 = rhist;  // its first 256 words are cleared every frame by the chore warp
      if (is_stay) {
        for (int i = tid; i < nb; i += NS) {
          const float sc = st_tot[i];
          if (sc > f_lo && !(sc > f_hi)) atomicAdd(&h2[sub_bin(sc)], 1u);
        }
      } else if (is_ext) {
        int q = q0, j = j0;
        for (int e = xl; e < next; e += NX) {
          const float sc = ext_score(hc[q], j);
          if (sc > f_lo && !(sc > f_hi) && !merged(e)) atomicAdd(&h2[sub_bin(sc)], 1u);
          step(q, j);
        }
      }
      __syncthreads();
      const Cut c2 = scan_score_histogram(h2, cut.left);
      sub_thr = c2.thr; sub_left = c2.left; sub_count = c2.cut_count;
      refined = c2.total > cut.left;  // always, unless NaN scores upset the counts
    }
    const bool take_all2 = refined && sub_count == sub_left;
    // 2: the candidate takes a beam slot, 1: it is in the (sub-)bin that the cut runs through,
    // 0: it is out
    auto klass = [&](float sc) -> int {
      if (sc > f_hi) return 2;
      if (!(sc > f_lo)) return 0;
      if (!kWide || !refined) return 1;
      const int sb = sub_bin(sc);
      if (sb < sub_thr || (take_all2 && sb == sub_thr)) return 2;
      return sb == sub_thr ? 1 : 0;
    };
    const int n_listed = refined ? (take_all2 ? 0 : sub_count) : (take_all ? 0 : cut.cut_count);
    const int n_winners = refined ? sub_left : cut.left;

    const bool fast_select = take_all || use_list || (refined && n_listed <= kListCap);  // block-uniform
    if (fast_select) {
      // P3a: every candidate above the cut bin takes a beam slot and is noted there; stays
      // fill the beam from slot 0 upwards, extensions from the last slot downwards.
      auto list_add = [&](unsigned key, int id) {
        const int li = atomicAdd(&sc_c[SC_LISTN], 1);
        if (li < kListCap) {
          list_key[li] = key;
          list_id[li] = id;
        }
      };
      if (is_stay && K <= NS && NS <= kOwnStayLanes && !kWide) {
        // Every beam entry has a stay lane of its own, in at most four stay warps: each looks at all (at most 128) stay candidates itself, so
        // the places follow from ballots alone and no counter is shared.
        int before = 0, total_sel = 0;  // selected stays in the warps below this one / in all
        float sc = neg_inf();
        int kl = 0;
        unsigned m_own = 0u;
#pragma unroll
        for (int w = 0; w < kOwnStayLanes / 32; ++w) {
          if (w * 32 < NS) {
            const float s_w = w * 32 + lane < nb ? st_tot[w * 32 + lane] : neg_inf();
            const int k_w = klass(s_w);
            const unsigned m_w = __ballot_sync(kFull, k_w == 2);
            const int n_w = __popc(m_w);
            before += w < warp ? n_w : 0;
            total_sel += n_w;
            if (w == warp) { sc = s_w; kl = k_w; m_own = m_w; }
          }
        }
        // a stay lane has no use for the extension-score registers: they carry its own
        // candidate and the slot it won over the barrier, and it writes it to the next beam itself
        int at = -1;
        if (kl == 2) at = before + __popc(m_own & lt_mask);
        kc[0] = sc;
        kc[1] = __int_as_float(at < K ? at : -1);
        if (tid == 0) sc_c[SC_SLOT] = total_sel;  // read after B3
        if (kl == 1) list_add(score_key(sc), tid << 16);
      } else if (is_stay) {
        // stays are dense: one ballot per round, the warp's places taken by its first lane
        for (int base = 0; base < nb; base += NS) {
          const int i = base + tid;
          const float sc = i < nb ? st_tot[i] : neg_inf();
          const int kl = klass(sc);
          const bool sel = kl == 2;
          const unsigned m = __ballot_sync(kFull, sel);
          if (m) {
            int at = 0;
            if (lane == 0) at = atomicAdd(&sc_c[SC_SLOT], __popc(m));
            at = __shfl_sync(kFull, at, 0) + __popc(m & lt_mask);
            if (sel && at < K) {
              sel_key[at] = score_key(sc);
              sel_id[at] = i << 16;
            }
          }
          if (kl == 1) list_add(score_key(sc), i << 16);
        }
      } else if (is_ext) {
        // extensions in the cut bin or above: the lanes of a warp that arrive here together
        // take their places with one atomic
        auto settle = [&](int e, int q, int j, float sc) {
          const int kl = klass(sc);
          if (kl == 0 || merged(e)) return;
          const unsigned key = score_key(sc);
          const int id = (q << 16) | (j + 1);
          const bool sure = kl == 2;
          const unsigned act = __activemask();
          const unsigned ms = __ballot_sync(act, sure);
          const unsigned mine = sure ? ms : (act & ~ms);
          int* const counter = sure ? &sc_c[SC_SLOT_E] : &sc_c[SC_LISTN];
          const int leader = __ffs(mine) - 1;
          int at = 0;
          if (lane == leader) at = atomicAdd(counter, __popc(mine));
          at = __shfl_sync(mine, at, leader) + __popc(mine & lt_mask);
          if (sure) {
            const int slot = nbn - 1 - at;
            if ((unsigned)slot < (unsigned)K) {
              sel_key[slot] = key;
              sel_id[slot] = id;
            }
          } else if (at < kListCap) {
            list_key[at] = key;
            list_id[at] = id;
          }
        };
        unsigned want = 0u;  // bit k: cached candidate k is in the cut bin or above
#pragma unroll
        for (int k = 0; k < kCache; ++k) want |= (kc[k] > f_lo ? 1u : 0u) << k;
        for (unsigned m = want; m; m &= m - 1) {
          const int k = __ffs(m) - 1;
          int q, j;
          nth(k, q, j);
          settle(xl + k * NX, q, j, k == 0 ? kc[0] : k == 1 ? kc[1] : k == 2 ? kc[2] : kc[3]);
        }
        // candidates beyond the cache are evaluated again
        if (kCache * NX < next) {
          int q, j;
          nth(kCache, q, j);
          for (int e = xl + kCache * NX; e < next; e += NX) {
            const float sc = ext_score(hc[q], j);
            if (sc > f_lo) settle(e, q, j, sc);
            step(q, j);
          }
        }
      } else if (kWideRows && fused() && V > kFusedMaxV) {
        // chore warp, while the others settle their candidates: the survivors of frame t+2 (by
        // now the counts have moved up a frame: it is the frame after the next)
        c1 = finish_wide_row();
      }
      clock_mark(4);
      __syncthreads();  // B3: every selected candidate is noted, the cut bin's members listed
      // P3b: one candidate per lane is written to the next beam; the chore warp meanwhile
      // ranks the members of the cut bin exactly (score, then candidate id) and writes the
      // winners to the slots between the stays and the extensions.
      const int n_stay = min(sc_c[SC_SLOT], K);
      if (is_stay && K <= NS && NS <= kOwnStayLanes && !kWide) {
        const int slot = __float_as_int(kc[1]);
        if (slot >= 0) place_stay(tid, score_key(kc[0]), slot);
      } else if (is_stay) {
        for (int s2 = tid; s2 < n_stay; s2 += NS) place_stay(sel_id[s2] >> 16, sel_key[s2], s2);
      } else if (is_ext) {
        const int n_ext = min(sc_c[SC_SLOT_E], K);
        for (int x = xl; x < n_ext; x += NX) {
          const int slot = nbn - 1 - x;
          if (slot >= 0) place_by_id(sel_id[slot], sel_key[slot], slot, x);
        }
      }
      // The members of the cut bin are ranked by (score, candidate id) and the best n_winners
      // go to the slots between the stays and the extensions.  All warps share the work: a warp
      // takes every NW-th member and counts, with one ballot per 32 members, how many beat it;
      // then one lane per winner writes it.  (The extensions among the winners are numbered
      // after those placed above.)
      if (n_listed > 0) {  // block-uniform
        const int n = min(n_listed, kListCap);
        const int n_ext = min(sc_c[SC_SLOT_E], K);
        const unsigned key_a = lane < n ? list_key[lane] : 0u;
        const int id_a = lane < n ? list_id[lane] : 0;
        const unsigned key_b = lane + 32 < n ? list_key[lane + 32] : 0u;
        const int id_b = lane + 32 < n ? list_id[lane + 32] : 0;
        int n_won = 0, my_m = -1, my_rank = 0;
        for (int m = warp; m < n; m += NW) {
          const unsigned key = list_key[m];
          const int id = list_id[m];
          int rank = __popc(__ballot_sync(kFull, lane < n && (key_a > key || (key_a == key && id_a < id))));
          if (n > 32)
            rank += __popc(__ballot_sync(
                kFull, lane + 32 < n && (key_b > key || (key_b == key && id_b < id))));
          if (rank < n_winners) {
            if (lane == n_won) { my_m = m; my_rank = rank; }
            ++n_won;
          }
        }
        if (n_won) {  // warp-uniform; lane i writes the i-th winner this warp found
          const bool mine = my_m >= 0;
          const int id = mine ? list_id[my_m] : 0;
          const unsigned mx = __ballot_sync(kFull, mine && (id & 0xffff) != 0);
          int base = 0;
          if (lane == 0 && mx) base = atomicAdd(&sc_c[SC_WIN_E], __popc(mx));
          base = __shfl_sync(kFull, base, 0);
          if (mine)
            place_by_id(id, list_key[my_m], n_stay + my_rank, n_ext + base + __popc(mx & lt_mask));
        }
      }
    } else {
      // ---- exact fallback: radix select over the integer keys ------------------------
      if (kWideRows && is_chore && fused() && V > kFusedMaxV) c1 = finish_wide_row();
      auto for_each_candidate = [&](auto&& f) {
        if (is_stay) {
          for (int i = tid; i < nb; i += NS) f(score_key(st_tot[i]), i << 16);
        } else if (is_ext) {
          int q = q0, j = j0;
          for (int e = xl; e < next; e += NX) {
            unsigned key = ext_key(hc[q], j);
            if (key && merged(e)) key = 0u;
            f(key, (q << 16) | (j + 1));
            step(q, j);
          }
        }
      };
      for (int i = tid; i < kPasses * kBins; i += NT) rhist[i] = 0u;
      if (tid == 0) {
        ++scal[SC_EXACT];  // frames that needed the exact select
        scal[SC_PREFIX] = 0; scal[SC_NEED] = K; scal[SC_DONE] = 0; scal[SC_TAKEALL] = 0;
        scal[SC_SHIFT] = 0; scal[SC_NBEAM_NEXT] = K;
      }
      __syncthreads();
      for (int pass = 0; pass < kPasses; ++pass) {
        const int sh = 32 - kRadixBits * (pass + 1);
        const unsigned prefix = (unsigned)scal[SC_PREFIX];
        unsigned* h = rhist + pass * kBins;
        for_each_candidate([&](unsigned key, int) {
          if (key && (pass == 0 || (key >> (sh + kRadixBits)) == prefix))
            atomicAdd(&h[(key >> sh) & (kBins - 1)], 1u);
        });
        __syncthreads();
        if (tid < 32) resolve_digit(h, scal, pass, sh);
        __syncthreads();
        if (scal[SC_DONE]) break;  // block-uniform
      }
      const int sh = scal[SC_SHIFT];
      const unsigned prefix = (unsigned)scal[SC_PREFIX];
      const int need = scal[SC_NEED];
      const bool r_all = scal[SC_TAKEALL] != 0;
      nbn = scal[SC_NBEAM_NEXT];
      unsigned long long mine = 0ull;
      for_each_candidate([&](unsigned key, int) {
        if (key) {
          const unsigned hk = key >> sh;
          mine += (hk > prefix) ? 1ull : ((hk == prefix) ? (1ull << 32) : 0ull);
        }
      });
      unsigned long long total;
      const unsigned long long excl = block_exclusive_scan(mine, warp_sums, &total);
      int gt_rank = (int)(excl & 0xffffffffull), eq_rank = (int)(excl >> 32);
      const int total_gt = (int)(total & 0xffffffffull);
      for_each_candidate([&](unsigned key, int id) {
        if (!key) return;
        const unsigned hk = key >> sh;
        int slot = -1;
        if (hk > prefix) {
          slot = gt_rank++;
        } else if (hk == prefix) {
          if (r_all || eq_rank < need) slot = total_gt + eq_rank;
          ++eq_rank;
        }
        if (slot >= 0) {
          int ord = 0;
          if (id & 0xffff) {
            // a new prefix: numbered through one shared counter, one atomic for all lanes of the
            // warp that are here together
            const unsigned here = __activemask();
            const int leader = __ffs(here) - 1;
            if (lane == leader) ord = atomicAdd(&sc_c[SC_SLOT_E], __popc(here));
            ord = __shfl_sync(here, ord, leader) + __popc(here & lt_mask);
          }
          place_by_id(id, key, slot, ord);
        }
      });
      __syncthreads();
      if (tid == 0) scal[SC_MADE + par] = sc_c[SC_SLOT_E];
    }
    if (cut.total == 0) status |= 8;  // FLTOP_ST_EMPTY_BEAM
    offset += (double)best;
    clock_mark(6);
    __syncthreads();  // B4: the next beam and its hash table are complete
    clock_mark(7);

    // (chore warp) what the next frame has to write out
    // new prefixes of the frame (they have consecutive node ids)
    const int made = min(fast_select ? min(sc_c[SC_SLOT_E], K) + sc_c[SC_WIN_E] : scal[SC_MADE + par], K);
    pend_at = n_nodes;
    pend_bytes = (arena_ok && made > 0) ? (unsigned)(((made + 1) & ~1) * sizeof(TrieNode)) : 0u;
    if (!arena_ok && made > 0) status |= 2;  // FLTOP_ST_ARENA_FULL
    if (arena_ok) n_nodes += (made + 1) & ~1;
    live_sum += nbn;
    nb = nbn;
    cur = nxt;
  }
  frames_seen += len;
  // the last frame's nodes; the read-out below walks the trie, so wait for all of them
  if (is_chore && lane == 0) {
    if (pend_bytes) bulk_store(nodes + pend_at, nstage + ((len - 1) & 1) * NSL, pend_bytes);
    bulk_store_wait_all();
  }
  __syncthreads();

  status |= scal[SC_STATUS];
  if (p.stats) {
    if (created) atomicAdd(&scal[SC_CREATED], created);
    if (tag_clashes) atomicAdd(&scal[SC_CLASHES], tag_clashes);
    __syncthreads();
    if (tid == 0) {
      int32_t* o = p.stats + kStatWords * (int64_t)b;
      o[0] = len; o[1] = scal[SC_CREATED]; o[2] = live_sum - scal[SC_DEAD]; o[3] = n_nodes;
      o[4] = scal[SC_CLASHES]; o[5] = scal[SC_EXACT];
      o[6] = scal[SC_KEPT];  // survivors, when this kernel pruned the frames itself
    }
  }

  const Hot* const hc = hot_base + cur * KS;
  const Ident* const id_c = ident_base + cur * KS;
  const Where* const wh_c = where_base + cur * KS;

  // ---- keep the beam for the next chunk (streaming) -----------------------------------
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
      hd->drift = 0;
    }
  }

  // ---- hypotheses, best first (GetHighestScorePrefix over the whole beam) ----------
  if (do_emit) {
    const int Lout = p.L;
    bool truncated = false;
    for (int i = tid; i < nb; i += NT) {
      const float ti = hc[i].tot;
      if (ti == neg_inf()) continue;  // a slot emptied by beam_threshold
      atomicAdd(&scal[SC_NLIVE], 1);
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
    if (truncated) atomicOr(&scal[SC_STATUS], 4);  // FLTOP_ST_TRUNCATED
    __syncthreads();
    const int n_live = scal[SC_NLIVE];
    for (int k = n_live + tid; k < K; k += NT) {
      p.out_lens[(int64_t)b * K + k] = 0;
      p.out_scores[(int64_t)b * K + k] = neg_inf();
    }
    status |= scal[SC_STATUS];
    if (tid == 0) p.out_nhyp[b] = n_live;
  }
  if (tid == 0 && p.out_status) p.out_status[b] = status;
}

}  // namespace

// Layout variants: small beams over a character or a subword vocabulary get compile-time
// array offsets, everything else the generic kernel.
enum Variant { kCharBeam64, kSubwordBeam64, kCharGeneric, kCharWideBeam, kGeneric, kWideBeam };
constexpr int kWideBeamFrom = 257;  // measured: the wide-beam devices pay off from here
Variant pick_variant(int K, int V) {
  if (K <= 64 && V <= 32) return kCharBeam64;
  if (K <= 64 && V <= 1024) return kSubwordBeam64;
  if (V <= 32) return K >= kWideBeamFrom ? kCharWideBeam : kCharGeneric;
  return K >= kWideBeamFrom ? kWideBeam : kGeneric;
}

size_t decode_smem_bytes(int K, int V) {
  switch (pick_variant(K, V)) {
    case kCharBeam64: return make_layout(64, 32).total;
    case kSubwordBeam64: return make_layout(64, 1024).total;
    case kCharGeneric:
    case kCharWideBeam: return make_layout(K, 32).total;
    default: return make_layout(K, V).total;
  }
}

int decode_block_threads(int K, int V, bool pruning, int top_n, bool latency_bound) {
  // One lane per beam entry for the stay candidates, one chore warp, and ext lanes for the
  // extension candidates: one candidate per lane, counting at most eight survivors per entry,
  // when every utterance has an SM to itself (the frame chain is all that matters); about
  // three per lane when blocks share SMs.  With pruning on, a quarter of a large vocabulary
  // (at least eight tokens) is assumed to survive a frame.
  long long cols = V;
  if (pruning) {
    cols = V / 4;
    if (cols < 8) cols = 8;
    if (cols > V) cols = V;
  }
  if (top_n > 0 && top_n < cols) cols = top_n;
  const long long stay = ((long long)K + 31) / 32 * 32;
  // (a character vocabulary: at most eight survivors per entry are counted; a wide one brings
  // hundreds of survivors a frame and wants every lane it can get)
  const long long per_entry = V > 32 ? cols : (cols < 8 ? cols : 8);
  long long ext = latency_bound ? (long long)K * per_entry : (long long)K * cols / 3;
  ext = (ext + 31) / 32 * 32;
  if (ext < 32) ext = 32;
  long long nt = stay + ext + 32;
  if (nt > kMaxThreads) nt = kMaxThreads;
  // A block of at most 512 threads has 128 registers a thread instead of 64; with pruning on
  // and a beam of moderate width that is worth more than the extra lanes (measured at V = 32:
  // 3 to 12 % faster for K = 64 ... 160, slower from K = 200).
  if (latency_bound && pruning && K <= 160 && V <= 32 && nt > kMidBlock) nt = kMidBlock;
  return (int)nt;
}

namespace {
template <int KMAX, int VMAX>
cudaError_t prepare_variant(int bytes) {
  const auto attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
  cudaError_t e = cudaFuncSetAttribute(decode_kernel<kSmallBlock, KMAX, VMAX, false>, attr, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_kernel<kMidBlock, KMAX, VMAX, false>, attr, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_kernel<kMaxThreads, KMAX, VMAX, false>, attr, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_kernel<kSmallBlock, KMAX, VMAX, true>, attr, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_kernel<kMidBlock, KMAX, VMAX, true>, attr, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_kernel<kMaxThreads, KMAX, VMAX, true>, attr, bytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(decode_kernel<kMaxThreads, KMAX, VMAX, false, true>, attr, bytes);
  return e;
}
template <int KMAX, int VMAX>
void launch_variant(const DecodeParams& p0, int nt, size_t bytes, bool alone, int sms, cudaStream_t s) {
  const bool bt = p0.beam_threshold > 0.f || p0.merge_max != 0;  // an option is on
  void (*kernel)(DecodeParams) = nullptr;
  if (nt <= kSmallBlock) {
    kernel = bt ? decode_kernel<kSmallBlock, KMAX, VMAX, true> : decode_kernel<kSmallBlock, KMAX, VMAX, false>;
  } else if (nt <= kMidBlock && alone) {
    // one block per SM: it may as well have 128 registers a thread (blocks that share an SM
    // keep to 64 so that two of 512 threads fit)
    kernel = bt ? decode_kernel<kMidBlock, KMAX, VMAX, true> : decode_kernel<kMidBlock, KMAX, VMAX, false>;
  } else {
    kernel = bt ? decode_kernel<kMaxThreads, KMAX, VMAX, true> : decode_kernel<kMaxThreads, KMAX, VMAX, false>;
  }
  // (phase clocks: the instrumented instantiation, whatever the block size)
  if (p0.dbg_clocks && !bt) kernel = decode_kernel<kMaxThreads, KMAX, VMAX, false, true>;
  DecodeParams p = p0;
  if (p.first_wave > 0) {
    // Blocks that all fit on the GPU at once: one per SM takes a long utterance, the ones that
    // move in beside them the short ones.  More blocks than fit: longest first throughout.
    int per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, nt, bytes) != cudaSuccess) {
      cudaGetLastError();
      per_sm = 1;
    }
    p.first_wave = (int64_t)p.B <= (int64_t)per_sm * sms ? sms : p.B;
  }
  kernel<<<p.B, nt, bytes, s>>>(p);
}
}  // namespace

bool decode_can_prune(int V, int dtype, const void* logp, int64_t stride_b, int64_t stride_t,
                      int top_n) {
  if (V > kFusedWideMaxV) return false;
  if (V > kFusedMaxV) {
    // wide rows are fetched 16 bytes at a time and walked by one warp: float32, rows that
    // start on a 16-byte boundary, no top-N stage (that is the cap kernel's radix select)
    return dtype == kEmissionF32 && (top_n <= 0 || top_n >= V) && V % 4 == 0 &&
           stride_b % 4 == 0 && stride_t % 4 == 0 && (reinterpret_cast<uintptr_t>(logp) & 15u) == 0;
  }
  if (dtype == kEmissionF32) return true;
  // two-byte elements are fetched in pairs: every row has to start on a four-byte boundary
  return V % 2 == 0 && stride_b % 2 == 0 && stride_t % 2 == 0 &&
         (reinterpret_cast<uintptr_t>(logp) & 3u) == 0;
}

cudaError_t decode_prepare(int K, int V) {
  const int bytes = (int)decode_smem_bytes(K, V);
  switch (pick_variant(K, V)) {
    case kCharBeam64: return prepare_variant<64, 32>(bytes);
    case kSubwordBeam64: return prepare_variant<64, 1024>(bytes);
    case kCharGeneric: return prepare_variant<0, 32>(bytes);
    case kCharWideBeam: return prepare_variant<-1, 32>(bytes);
    case kWideBeam: return prepare_variant<-1, 0>(bytes);
    default: return prepare_variant<0, 0>(bytes);
  }
}

cudaError_t launch_decode(const DecodeParams& p, cudaStream_t s) {
  if (p.B == 0) return cudaSuccess;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int blocks = p.co_resident > p.B ? p.co_resident : p.B;
  int nt = p.block_threads > 0
               ? p.block_threads
               : decode_block_threads(p.K, p.V, p.pruning != 0, p.top_n, blocks <= sms);
  if (p.block_threads <= 0 && nt > 512 && p.pruning && blocks > 2 * sms) {
    // many more utterances than SMs: what counts is throughput, and two blocks of 512 threads
    // per SM overlap their frame chains better than one block of 1024.  (Up to two blocks per
    // SM the launch lasts as long as its longest chains, which blocks of 1024 threads, started
    // longest first, finish sooner: 4.5 against 5.1 ms on 256 utterances of 1024 tokens.)
    nt = 512;
  }
  nt = (nt + 31) / 32 * 32;
  if (nt < 96) nt = 96;  // a stay warp, an ext warp and the chore warp
  if (nt > kMaxThreads) nt = kMaxThreads;
  const size_t bytes = decode_smem_bytes(p.K, p.V);
  DecodeParams q = p;
  // more utterances of one batch than SMs: the blocks take them by length
  q.first_wave = (!p.streaming && p.co_resident == 0 && p.B > sms && p.B <= kByLengthMaxB &&
                  bytes >= (size_t)(p.B + 1) * sizeof(int))
                     ? sms : 0;
  switch (pick_variant(p.K, p.V)) {
    case kCharBeam64: launch_variant<64, 32>(q, nt, bytes, blocks <= sms, sms, s); break;
    case kSubwordBeam64: launch_variant<64, 1024>(q, nt, bytes, blocks <= sms, sms, s); break;
    case kCharGeneric: launch_variant<0, 32>(q, nt, bytes, blocks <= sms, sms, s); break;
    case kCharWideBeam: launch_variant<-1, 32>(q, nt, bytes, blocks <= sms, sms, s); break;
    case kWideBeam: launch_variant<-1, 0>(q, nt, bytes, blocks <= sms, sms, s); break;
    default: launch_variant<0, 0>(q, nt, bytes, blocks <= sms, sms, s); break;
  }
  return cudaGetLastError();
}

}  // namespace fltop
