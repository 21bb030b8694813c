// CTC prefix beam search over pruned frames for narrow beams: one WARP per utterance.
//
// The block kernel (fltop_decode.cu) spends most of a frame on what a thread block needs to
// work together - four barriers, a histogram scan that the other warps wait for, counters
// shared through atomics - and that cost does not shrink with the beam: a frame of a
// 10-entry beam with a dozen candidates takes three quarters of the time of a 50-entry one.
// Here a beam of at most 32 entries over a vocabulary of at most 32 tokens lives in the
// registers of one warp, lane i holding beam entry i and (for the emission row) token i.
// Nothing waits for anything but the warp itself, several utterances share a block, and an
// SM runs as many utterances side by side as it has warp slots.
//
// The computation is the block kernel's, step for step (Algorithm 1 with the standard CTC
// collapsing rule):
//   prune    row maximum by a warp reduction, threshold by one float32 add, survivors as a
//            32-bit mask; the top-N stage lets the best remaining token leave N times.
//   extend   lane i evaluates "entry i stays"; for every surviving non-blank token (a loop
//            over the mask, the same for all lanes) lane i evaluates "entry i extended by it".
//   merge    an entry and its parent's extension by the entry's last token name the same
//            prefix: the entry finds its parent through a small table of the beam's 64-bit
//            sequence fingerprints, takes the extension's mass and marks it as merged.
//   select   the 256-bin score histogram and its warp scan give the cut; candidates above
//            the cut bin are placed at once, the members of the cut bin are ranked exactly.
//            When more than 64 candidates share the cut bin (near-equal scores) the K-th
//            best key is searched bit by bit instead.
//   trie     8-byte back-pointer records, one per new prefix, written when it enters the beam.
// Scores are relative to a per-frame reference summed in float64, as in the block kernel.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "fltop_device.cuh"
#include "fltop_internal.h"

namespace fltop {
namespace {

constexpr int kWarpsPerBlock = 4;  // utterances per block
constexpr int kWarpTab = 128;      // slots of the fingerprint table (four per beam entry)
constexpr unsigned kFree = 0xffffffffu;

// A beam as the warp keeps it in shared memory, next to the copy in its registers: whoever
// places a candidate into the next beam reads its source entry from here.
struct BeamCopy {
  int last[32];
  float pb[32], pnb[32], tot[32];
  unsigned long long print[32], pprint[32];
  int node[32], len[32];
};

struct WarpScratch {
  unsigned hist[kFastBins];
  unsigned tab[kWarpTab];
  unsigned dupw[32];           // bit c of word q: "entry q extended by token c" is merged
  unsigned list_key[kListCap];
  int list_id[kListCap];
  float st_pb[32], st_pnb[32]; // the stay candidate of every entry
  BeamCopy beam[2];
};

__device__ __forceinline__ float load_emission(const void* base, int dtype, int64_t at) {
  if (dtype == kEmissionF32) return static_cast<const float*>(base)[at];
  if (dtype == kEmissionF16) return __half2float(static_cast<const __half*>(base)[at]);
  return __bfloat162float(static_cast<const __nv_bfloat16*>(base)[at]);
}

__global__ void __launch_bounds__(32 * kWarpsPerBlock) decode_warp_kernel(DecodeParams p) {
  __shared__ __align__(16) WarpScratch scratch[kWarpsPerBlock];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int b = blockIdx.x * kWarpsPerBlock + warp;
  if (b >= p.B) return;  // the whole warp
  WarpScratch& S = scratch[warp];
  const int K = p.K, V = p.V, blank = p.blank;
  const unsigned lt_mask = (1u << lane) - 1u;

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
  int32_t* const st = p.streaming
                          ? p.state + (int64_t)b * (kStateHeaderWords + kStateWordsPerSlot * (int64_t)K)
                          : nullptr;

  // ---- the beam: lane i holds entry i ---------------------------------------------------
  int e_last = -1, e_node = 0, e_len = 0;
  float e_pb = neg_inf(), e_pnb = neg_inf(), e_tot = neg_inf();
  unsigned long long e_print = 0ull, e_pprint = 0ull;
  int nb, n_nodes, frames_seen;
  double offset;
  if (do_reset) {
    nb = bad_len && !p.streaming ? 0 : 1;
    n_nodes = 2;  // node 0 is the empty prefix; blocks of ids start even (as in the block kernel)
    offset = 0.0;
    frames_seen = 0;
    if (lane == 0) {
      e_pb = 0.f; e_tot = 0.f; e_print = kRootPrint;
      nodes[0] = TrieNode{-1, -1};
    }
  } else {
    const StateHeader* hd = reinterpret_cast<const StateHeader*>(st);
    nb = hd->nbeam; n_nodes = hd->n_nodes; frames_seen = hd->frames; offset = hd->offset;
    status |= hd->status;
    const int32_t* a = st + kStateHeaderWords;
    if (lane < nb) {
      e_node = a[lane]; e_last = a[K + lane]; e_len = a[2 * K + lane];
      e_pb = __int_as_float(a[3 * K + lane]);
      e_pnb = __int_as_float(a[4 * K + lane]);
      e_tot = __int_as_float(a[5 * K + lane]);
      e_print = reinterpret_cast<const unsigned long long*>(a + 6 * K)[lane];
      e_pprint = reinterpret_cast<const unsigned long long*>(a + 8 * K)[lane];
    }
  }
  int cur = 0;
  auto publish_beam = [&](BeamCopy& c) {  // registers -> shared copy (all lanes; unused slots too)
    c.last[lane] = e_last; c.pb[lane] = e_pb; c.pnb[lane] = e_pnb; c.tot[lane] = e_tot;
    c.print[lane] = e_print; c.pprint[lane] = e_pprint; c.node[lane] = e_node; c.len[lane] = e_len;
  };
  // Table of the beam's fingerprints: entries [tag : 20 | slot : 12], linear probing, never
  // more than a quarter full.
  auto rebuild_table = [&](int n) {  // from the fingerprints in the registers
    reinterpret_cast<uint4*>(S.tab)[lane] = make_uint4(kFree, kFree, kFree, kFree);
    __syncwarp();
    if (lane < n) {
      const unsigned long long h = e_print;
      const unsigned val = (((unsigned)h & 0xfffffu) << 12) | (unsigned)lane;
      const unsigned home = (unsigned)(h >> 40) & (kWarpTab - 1);
      unsigned pos = home;
      bool in = false;
      do {  // (ends at the latest back at its first slot)
        in = atomicCAS(&S.tab[pos], kFree, val) == kFree;
        pos = (pos + 1) & (kWarpTab - 1);
      } while (!in && pos != home);
      if (!in) status |= 16;  // FLTOP_ST_INTERNAL (cannot happen: 32 entries, 128 slots)
    }
  };
  auto table_find = [&](const BeamCopy& c, unsigned long long h) -> int {
    const unsigned tag = (unsigned)h & 0xfffffu;
    const unsigned home = (unsigned)(h >> 40) & (kWarpTab - 1);
    unsigned pos = home;
    do {
      const unsigned v = S.tab[pos];
      if (v == kFree) return -1;
      if ((v >> 12) == tag && c.print[v & 0xfffu] == h) return (int)(v & 0xfffu);
      pos = (pos + 1) & (kWarpTab - 1);
    } while (pos != home);
    return -1;
  };
  auto clear_frame_scratch = [&]() {
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    reinterpret_cast<uint4*>(S.hist)[2 * lane] = zero;
    reinterpret_cast<uint4*>(S.hist)[2 * lane + 1] = zero;
    S.dupw[lane] = 0u;
  };
  publish_beam(S.beam[cur]);
  clear_frame_scratch();
  __syncwarp();
  rebuild_table(nb);
  __syncwarp();

  const int64_t row0 = (int64_t)b * p.stride_b;
  float lp_next = neg_inf();
  if (len > 0 && lane < V) lp_next = load_emission(p.logp, p.dtype, row0 + lane);
  int kept_sum = 0, created = 0, live_sum = 0;

  for (int t = 0; t < len; ++t) {
    const BeamCopy& C = S.beam[cur];
    BeamCopy& N = S.beam[cur ^ 1];
    const float lp = lp_next;
    if (t + 1 < len && lane < V)
      lp_next = load_emission(p.logp, p.dtype, row0 + (int64_t)(t + 1) * p.stride_t + lane);

    // ---- prune: survivors of the frame as a mask over tokens ------------------------------
    const unsigned lu = __float_as_uint(lp);
    const unsigned okey = (lp == lp) ? ((lu & 0x80000000u) ? ~lu : (lu | 0x80000000u)) : 0x007fffffu;
    const unsigned mkey = __reduce_max_sync(kFull, okey);
    const float row_max = __uint_as_float((mkey & 0x80000000u) ? (mkey & 0x7fffffffu) : ~mkey);
    const float thr = __fadd_rn(row_max, p.log_r);
    const bool keep = lane < V && lp >= thr;
    unsigned kept = __ballot_sync(kFull, keep);
    if (p.top_n > 0 && __popc(kept) > p.top_n) {
      unsigned key = keep ? okey : 0u;  // 0 = not (or no longer) in the running
      unsigned chosen = 0u;
      for (int i = 0; i < p.top_n; ++i) {
        const unsigned best_key = __reduce_max_sync(kFull, key);
        const int w = __ffs(__ballot_sync(kFull, key == best_key)) - 1;  // ties: lower token id
        chosen |= 1u << w;
        if (lane == w) key = 0u;
      }
      kept = chosen;
    }
    kept_sum += __popc(kept);
    if (p.dbg_masks && lane == 0) p.dbg_masks[(int64_t)b * p.T + t] = kept;  // instrumented launches only
    const bool blank_kept = (kept >> blank) & 1u;
    const float lp_blank_raw = __shfl_sync(kFull, lp, blank);
    const float lp_blank = blank_kept ? lp_blank_raw : neg_inf();
    const unsigned kb = kept & ~(1u << blank);  // surviving non-blank tokens

    // ---- every candidate is evaluated once and counted ---------------------------------
    const float le_raw = __shfl_sync(kFull, lp, e_last < 0 ? 0 : e_last);
    float npb = neg_inf(), npnb = neg_inf(), stot = neg_inf();
    if (lane < nb) {
      npb = e_tot + lp_blank;
      float own = neg_inf(), dup = neg_inf();
      if (e_last >= 0) {
        const float le = ((kept >> e_last) & 1u) ? le_raw : neg_inf();
        own = e_pnb + le;
        const int pq = table_find(C, e_pprint);
        if (pq >= 0) {
          dup = ((C.last[pq] == e_last) ? C.pb[pq] : C.tot[pq]) + le;
          if (dup != neg_inf()) {  // the parent's extension by last(i) names this prefix
            atomicSub(&S.hist[score_bin(dup)], 1u);
            atomicOr(&S.dupw[pq], 1u << e_last);
          }
        }
      }
      npnb = lse2(own, dup);
      stot = lse3(npb, own, dup);
      if (stot != neg_inf()) atomicAdd(&S.hist[score_bin(stot)], 1u);
    }
    S.st_pb[lane] = npb;
    S.st_pnb[lane] = npnb;
    // score of "entry `lane` extended by token c" (c the same for all lanes)
    auto ext_score = [&](int c, float lc) -> float {
      if (lane >= nb) return neg_inf();
      return ((c == e_last) ? e_pb : e_tot) + lc;
    };
    for (unsigned m = kb; m; m &= m - 1) {
      const int c = __ffs(m) - 1;
      const float sc = ext_score(c, __shfl_sync(kFull, lp, c));
      if (sc != neg_inf()) atomicAdd(&S.hist[score_bin(sc)], 1u);
    }
    __syncwarp();

    // ---- the cut ------------------------------------------------------------------------
    const Cut cut = scan_score_histogram(S.hist, K);
    const float best = -(float)(cut.first * kBinsPerLane) * (1.f / kBinsPerNat);
    const bool take_all = cut.cut_count == cut.left;  // also when there is no cut at all
    const int nbn = min(cut.total, K);
    int n_new = 0;  // new prefixes of this frame so far
    const bool arena_ok = (int64_t)n_nodes + ((K + 1) & ~1) <= p.nodes_per_utt;
    const unsigned my_dup = S.dupw[lane];

    // Writing a candidate into slot `slot` of the next beam: c_plus1 = 0 stays as it is,
    // c_plus1 > 0 (token + 1) is a new prefix and gets its trie record; `ord` numbers the new
    // prefixes of the frame, which get consecutive node ids.
    auto place = [&](int q, int c_plus1, float sc, int slot, int ord) {
      if ((unsigned)slot >= (unsigned)K || (unsigned)ord >= (unsigned)K) return;  // (NaN scores)
      if (c_plus1 == 0) {
        N.last[slot] = C.last[q];
        N.pb[slot] = S.st_pb[q] - best;
        N.pnb[slot] = S.st_pnb[q] - best;
        N.tot[slot] = sc - best;
        N.print[slot] = C.print[q];
        N.pprint[slot] = C.pprint[q];
        N.node[slot] = C.node[q];
        N.len[slot] = C.len[q];
      } else {
        const int c = c_plus1 - 1;
        const unsigned long long pp = C.print[q];
        N.last[slot] = c;
        N.pb[slot] = neg_inf();
        N.pnb[slot] = sc - best;
        N.tot[slot] = sc - best;
        N.print[slot] = child_print(pp, c);
        N.pprint[slot] = pp;
        N.node[slot] = arena_ok ? n_nodes + ord : 0;  // arena full: nothing to walk back to
        N.len[slot] = C.len[q] + 1;
        if (arena_ok) nodes[n_nodes + ord] = TrieNode{C.node[q], c};
        ++created;
      }
    };

    // the same for the lane that owns the source entry: everything is in its registers
    auto place_own_stay = [&](int slot) {
      if ((unsigned)slot >= (unsigned)K) return;
      N.last[slot] = e_last;
      N.pb[slot] = npb - best;
      N.pnb[slot] = npnb - best;
      N.tot[slot] = stot - best;
      N.print[slot] = e_print;
      N.pprint[slot] = e_pprint;
      N.node[slot] = e_node;
      N.len[slot] = e_len;
    };
    auto place_own_ext = [&](int c, float sc, int slot, int ord) {
      if ((unsigned)slot >= (unsigned)K || (unsigned)ord >= (unsigned)K) return;
      N.last[slot] = c;
      N.pb[slot] = neg_inf();
      N.pnb[slot] = sc - best;
      N.tot[slot] = sc - best;
      N.print[slot] = child_print(e_print, c);
      N.pprint[slot] = e_print;
      N.node[slot] = arena_ok ? n_nodes + ord : 0;
      N.len[slot] = e_len + 1;
      if (arena_ok) nodes[n_nodes + ord] = TrieNode{e_node, c};
      ++created;
    };

    if (take_all || cut.cut_count <= kListCap) {
      // the cut as scores (bin edges): > f_hi is above the cut bin, > f_lo in it or above
      const float f_lo = (cut.thr >= kFastBins - 1) ? neg_inf()
                                                    : -(float)(cut.thr + 1) * (1.f / kBinsPerNat);
      const float f_hi = take_all ? f_lo
                                  : (cut.thr == 0 ? __int_as_float(0x7f800000)
                                                  : -(float)cut.thr * (1.f / kBinsPerNat));
      int n_list = 0, n_ext = 0;
      // stays take slots from 0 upwards
      const bool s_sure = stot > f_hi, s_list = !s_sure && stot > f_lo;
      const unsigned bs = __ballot_sync(kFull, s_sure);
      const int n_stay = __popc(bs);
      if (s_sure) place_own_stay(__popc(bs & lt_mask));
      {
        const unsigned bl = __ballot_sync(kFull, s_list);
        if (s_list) {
          const int li = __popc(bl & lt_mask);
          S.list_key[li] = score_key(stot);
          S.list_id[li] = lane << 16;
        }
        n_list = __popc(bl);
      }
      // extensions from the last slot downwards
      for (unsigned m = kb; m; m &= m - 1) {
        const int c = __ffs(m) - 1;
        float sc = ext_score(c, __shfl_sync(kFull, lp, c));
        if ((my_dup >> c) & 1u) sc = neg_inf();  // merged into a stay candidate
        const bool x_sure = sc > f_hi, x_list = !x_sure && sc > f_lo;
        const unsigned bx = __ballot_sync(kFull, x_sure);
        if (x_sure) {
          const int ord = n_ext + __popc(bx & lt_mask);
          place_own_ext(c, sc, nbn - 1 - ord, ord);
        }
        n_ext += __popc(bx);
        const unsigned bl = __ballot_sync(kFull, x_list);
        if (x_list) {
          const int li = n_list + __popc(bl & lt_mask);
          if (li < kListCap) {
            S.list_key[li] = score_key(sc);
            S.list_id[li] = (lane << 16) | (c + 1);
          }
        }
        n_list += __popc(bl);
      }
      __syncwarp();
      // the members of the cut bin, ranked by (score, candidate id): the best `left` go in between
      n_new = n_ext;
      if (!take_all) {
        const int n = min(n_list, kListCap);
        for (int base = 0; base < n; base += 32) {
          const int li = base + lane;
          unsigned key = 0u;
          int id = 0, rank = 0x7fffffff;
          if (li < n) {
            key = S.list_key[li];
            id = S.list_id[li];
            rank = 0;
            for (int j = 0; j < n; ++j) {
              const unsigned kj = S.list_key[j];
              rank += (kj > key || (kj == key && S.list_id[j] < id)) ? 1 : 0;
            }
          }
          const bool won = rank < cut.left;
          const unsigned mx = __ballot_sync(kFull, won && (id & 0xffff) != 0);
          if (won)
            place(id >> 16, id & 0xffff, key_score(key), n_stay + rank,
                  n_new + __popc(mx & lt_mask));
          n_new += __popc(mx);
        }
      }
    } else {
      // Crowded cut bin: the K-th best key, bit by bit (each step counts the candidates whose
      // key is at least the trial value), then everything above it and, in candidate order,
      // as many of its equals as are still needed.
      const unsigned s_key = score_key(stot);
      unsigned kth = 0u;
      for (int bit = 31; bit >= 0; --bit) {
        const unsigned trial = kth | (1u << bit);
        int cnt = __popc(__ballot_sync(kFull, s_key >= trial));
        for (unsigned m = kb; m; m &= m - 1) {
          const int c = __ffs(m) - 1;
          float sc = ext_score(c, __shfl_sync(kFull, lp, c));
          if ((my_dup >> c) & 1u) sc = neg_inf();
          cnt += __popc(__ballot_sync(kFull, score_key(sc) >= trial));
        }
        if (cnt >= K) kth = trial;
      }
      // pass 1: how many are above the K-th key
      int n_above_stay = __popc(__ballot_sync(kFull, s_key > kth)), n_above = n_above_stay;
      for (unsigned m = kb; m; m &= m - 1) {
        const int c = __ffs(m) - 1;
        float sc = ext_score(c, __shfl_sync(kFull, lp, c));
        if ((my_dup >> c) & 1u) sc = neg_inf();
        n_above += __popc(__ballot_sync(kFull, score_key(sc) > kth));
      }
      int need = K - n_above;  // equals of the K-th key still to take (at least one)
      // pass 2: placement; ties go to the slots after the stays, in candidate order
      int n_ext = 0, n_tie = 0;
      {
        const bool above = s_key > kth, tie = s_key == kth && kth != 0u;
        const unsigned ba = __ballot_sync(kFull, above);
        if (above) place_own_stay(__popc(ba & lt_mask));
        const unsigned bt = __ballot_sync(kFull, tie);
        const int r = __popc(bt & lt_mask);
        if (tie && r < need) place_own_stay(n_above_stay + r);
        n_tie += min(__popc(bt), need);
      }
      for (unsigned m = kb; m; m &= m - 1) {
        const int c = __ffs(m) - 1;
        float sc = ext_score(c, __shfl_sync(kFull, lp, c));
        if ((my_dup >> c) & 1u) sc = neg_inf();
        const unsigned key = score_key(sc);
        const bool above = key > kth, tie = key == kth && kth != 0u;
        const unsigned ba = __ballot_sync(kFull, above);
        if (above) place_own_ext(c, sc, nbn - 1 - (n_ext + __popc(ba & lt_mask)),
                                 n_new + __popc(ba & lt_mask));
        n_ext += __popc(ba);
        n_new += __popc(ba);
        const unsigned bt = __ballot_sync(kFull, tie);
        const int r = n_tie + __popc(bt & lt_mask);
        const unsigned taken = __ballot_sync(kFull, tie && r < need);
        if (tie && r < need) place_own_ext(c, sc, n_above_stay + r, n_new + __popc(taken & lt_mask));
        n_new += __popc(taken);
        n_tie = min(n_tie + __popc(bt), need);
      }
    }
    if (cut.total == 0) status |= 8;  // FLTOP_ST_EMPTY_BEAM
    if (!arena_ok && n_new > 0) status |= 2;  // FLTOP_ST_ARENA_FULL
    __syncwarp();

    // ---- the next beam becomes the beam -----------------------------------------------------
    e_last = -1; e_node = 0; e_len = 0;
    e_pb = e_pnb = e_tot = neg_inf();
    e_print = e_pprint = 0ull;
    if (lane < nbn) {
      e_last = N.last[lane]; e_pb = N.pb[lane]; e_pnb = N.pnb[lane]; e_tot = N.tot[lane];
      e_print = N.print[lane]; e_pprint = N.pprint[lane]; e_node = N.node[lane]; e_len = N.len[lane];
    }
    offset += (double)best;
    if (arena_ok) n_nodes += (n_new + 1) & ~1;
    live_sum += nbn;
    nb = nbn;
    cur ^= 1;
    clear_frame_scratch();
    rebuild_table(nb);
    __syncwarp();
  }
  frames_seen += len;
  status = (int)__reduce_or_sync(kFull, (unsigned)status);  // a lane's flag is the warp's

  // (survivors are not listed per frame: their total goes out with the statistics)
  if (p.stats) {
    const int made = __reduce_add_sync(kFull, created);
    if (lane == 0) {
      int32_t* o = p.stats + kStatWords * (int64_t)b;
      o[0] = len; o[1] = made; o[2] = live_sum; o[3] = n_nodes; o[4] = 0; o[5] = 0;
      o[6] = kept_sum;
    }
  }

  // ---- keep the beam for the next chunk (streaming) -----------------------------------------
  if (p.streaming) {
    int32_t* a = st + kStateHeaderWords;
    if (lane < nb) {
      a[lane] = e_node; a[K + lane] = e_last; a[2 * K + lane] = e_len;
      a[3 * K + lane] = __float_as_int(e_pb); a[4 * K + lane] = __float_as_int(e_pnb);
      a[5 * K + lane] = __float_as_int(e_tot);
      reinterpret_cast<unsigned long long*>(a + 6 * K)[lane] = e_print;
      reinterpret_cast<unsigned long long*>(a + 8 * K)[lane] = e_pprint;
    }
    if (lane == 0) {
      StateHeader* hd = reinterpret_cast<StateHeader*>(st);
      hd->nbeam = nb; hd->n_nodes = n_nodes; hd->frames = frames_seen;
      hd->status = status & ~1;  // a bad chunk length is not sticky
      hd->offset = offset;
      hd->drift = 0;
    }
  }

  // ---- hypotheses, best first -------------------------------------------------------------------
  if (do_emit) {
    // the trie records of this call were written by other lanes of this warp
    __threadfence_block();
    __syncwarp();
    int rank = 0;
    for (int j = 0; j < nb; ++j) {
      const float tj = __shfl_sync(kFull, e_tot, j);
      rank += (tj > e_tot || (tj == e_tot && j < lane)) ? 1 : 0;
    }
    bool truncated = false;
    if (lane < nb) {
      const int Lout = p.L;
      const int64_t o = (int64_t)b * K + rank;
      p.out_scores[o] = (float)(offset + (double)e_tot);
      p.out_lens[o] = e_len;
      if (e_len > Lout) truncated = true;
      int32_t* dst = p.out_tokens + o * Lout;
      int node = e_node;
      for (int d = e_len - 1; d >= 0 && node > 0 && (int64_t)node < p.nodes_per_utt; --d) {
        const int2 rec = *reinterpret_cast<const int2*>(&nodes[node]);  // parent, token
        if (d < Lout) dst[d] = rec.y;
        node = rec.x;
      }
    }
    if (__any_sync(kFull, truncated)) status |= 4;  // FLTOP_ST_TRUNCATED
    for (int k = nb + lane; k < K; k += 32) {
      p.out_lens[(int64_t)b * K + k] = 0;
      p.out_scores[(int64_t)b * K + k] = neg_inf();
    }
    if (lane == 0) p.out_nhyp[b] = nb;
  }
  if (lane == 0 && p.out_status) p.out_status[b] = status;
}

}  // namespace

bool decode_warp_eligible(const DecodeParams& p) {
  // narrow beam, one token per lane, the rows at hand, none of the options of the block
  // kernel's own instantiations, and no block size asked for
  const bool can = p.K <= 32 && p.V <= 32 && p.logp != nullptr && !(p.beam_threshold > 0.f) &&
                   p.merge_max == 0 && p.block_threads <= 0;
  if (!can || p.warp_mode == 0) return false;
  if (p.warp_mode == 2) return true;
  // A warp alone walks a frame more slowly than a block does (measured, K = 16, three
  // survivors a frame: 5.7 us against 3.2 us with seven blocks to an SM), but an SM holds
  // many more of them: it pays once utterances outnumber the SMs about eight to one
  // (1536 streams: 91 against 113 us per 16-frame chunk; 16384 streams: 293 against 1009 us).
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  return p.B >= 8 * sms;
}

cudaError_t launch_decode_warp(const DecodeParams& p, cudaStream_t s) {
  if (p.B == 0) return cudaSuccess;
  const int blocks = (p.B + kWarpsPerBlock - 1) / kWarpsPerBlock;
  decode_warp_kernel<<<blocks, 32 * kWarpsPerBlock, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace fltop
