// CPU oracle for frame-pruned CTC prefix beam search.  TEST INFRASTRUCTURE ONLY.
//
// This file is the slow, single-threaded, plainly written statement of what
// the decoder computes.  It exists so that tests (and the benchmark's CPU
// baseline leg) have something to compare the CUDA library with; the product
// never calls it, and it shares no code with the CUDA sources.
//
// What it follows (paper: "FLToP CTC", Algorithm 1 and Section 3):
//   * beam initialised with the empty prefix at log-score 0      (Alg. 1, init)
//   * for every frame, tokens are kept only if their probability is at least
//     R times the frame's top probability (Alg. 1, the conditional break;
//     Section 3 "relative threshold R times the highest score").  With
//     log-probabilities this is  lp >= lp_max + log R, evaluated in float32
//     with one float32 addition, exactly as stated here.
//   * every beam entry is extended by every surviving token    (Alg. 1, loops)
//   * candidates naming the same prefix are combined, the best beam_size are
//     kept (Alg. 1, B'.add and SelectTopK)
//   * after the last frame the prefixes are returned best first (Alg. 1,
//     GetHighestScorePrefix, widened to the whole beam).
// Algorithm 1 leaves out the CTC collapsing rule of the "standard
// BeamSearchCTC decoders" it modifies (Section 3); the standard rule is used:
// every prefix carries the log-mass of its alignments ending in blank (pb) and
// ending in its last token (pnb).  The language model of Algorithm 1 is not part
// of this path.  The two remaining knobs of Algorithm 1 are optional:
//   * N (PartialSortDesc(logits[t], N)): only the N most probable tokens of a
//     frame are considered at all, before the relative threshold is applied;
//     at a tie for the N-th place the lower token id wins.  top_n = 0 means N = V.
//   * beam_threshold (second argument of SelectTopK): after the best beam_size
//     candidates are chosen, those scoring below best - beam_threshold are
//     dropped.  beam_threshold <= 0 means no such cut.
// A third option restates Algorithm 1's score update literally: it writes
// score' = score + logit for a candidate and never sums over the alignments
// of a prefix, which is what decoders of the flashlight family do when their
// log-add option is off.  With merge_max every combination of two masses
// below (equal prefixes in B'.add, blank and non-blank mass of a prefix) takes
// the larger one, so a prefix's score is that of its single best alignment.
//
// A prefix is identified by its full token sequence.  Sequences are stored in
// a trie whose child table is never pruned, so one node id corresponds to
// exactly one sequence for the life of an utterance.
//
// Scores are float64.  The prune comparison is float32 (compile with
// -ffp-contract=off so that the single addition is not fused).
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <map>
#include <utility>
#include <vector>

namespace {

const double NEG_INF = -std::numeric_limits<double>::infinity();

double log_add(double a, double b) {
  if (a == NEG_INF) return b;
  if (b == NEG_INF) return a;
  double hi = a > b ? a : b, lo = a > b ? b : a;
  return hi + std::log1p(std::exp(lo - hi));
}

struct Mass {
  double pb = NEG_INF;   // log-mass of alignments of this prefix ending in blank
  double pnb = NEG_INF;  // ... ending in the prefix's last token
};

struct TrieNode {
  int parent;
  int token;
  int depth;
};

struct Decoder {
  int V, blank, K;
  int top_n = 0;                 // 0: no cap
  double beam_threshold = 0.0;   // <= 0: no cut
  bool merge_max = false;        // combine masses by max instead of log-sum
  float log_r;
  std::vector<TrieNode> nodes;                  // node 0 = empty prefix
  std::map<std::pair<int, int>, int> child;     // (parent node, token) -> node
  std::vector<std::pair<int, Mass>> beam;       // (node id, mass), best first
  int64_t frames_seen = 0;

  Decoder(int V_, int blank_, int K_, float r) : V(V_), blank(blank_), K(K_) {
    // log R once, in double, rounded to float32; R = 0 gives -inf (no pruning)
    log_r = r > 0.f ? (float)std::log((double)r) : -std::numeric_limits<float>::infinity();
    reset();
  }

  void reset() {
    nodes.assign(1, TrieNode{-1, -1, 0});
    child.clear();
    Mass m;
    m.pb = 0.0;  // the empty prefix has probability 1 before any frame
    beam.assign(1, std::make_pair(0, m));
    frames_seen = 0;
  }

  double combine(double a, double b) const { return merge_max ? std::max(a, b) : log_add(a, b); }
  double total(const Mass& m) const { return combine(m.pb, m.pnb); }

  int child_of(int p, int c) {
    auto key = std::make_pair(p, c);
    auto it = child.find(key);
    if (it != child.end()) return it->second;
    int id = (int)nodes.size();
    nodes.push_back(TrieNode{p, c, nodes[p].depth + 1});
    child.emplace(key, id);
    return id;
  }

  std::vector<int> sequence(int node) const {
    std::vector<int> s(nodes[node].depth);
    for (int n = node; n > 0; n = nodes[n].parent) s[nodes[n].depth - 1] = nodes[n].token;
    return s;
  }

  // Frame-level pruning: the survivor set of one frame.
  // keep[c] = (lp[c] >= max + log_r) in float32.
  int prune(const float* lp, uint8_t* keep) const {
    float m = lp[0];
    for (int c = 1; c < V; ++c)
      if (lp[c] > m) m = lp[c];
    volatile float thr = m + log_r;  // one rounded float32 addition
    int n = 0;
    for (int c = 0; c < V; ++c) {
      keep[c] = lp[c] >= thr ? 1 : 0;
      n += keep[c];
    }
    if (top_n > 0 && n > top_n) {
      // stage 1 of Algorithm 1: only the top_n most probable tokens are looked at
      std::vector<int> order;
      for (int c = 0; c < V; ++c)
        if (keep[c]) order.push_back(c);
      std::stable_sort(order.begin(), order.end(),
                       [lp](int a, int b) { return lp[a] > lp[b]; });  // ties keep id order
      for (size_t i = top_n; i < order.size(); ++i) keep[order[i]] = 0;
      n = top_n;
    }
    return n;
  }

  void step(const float* lp, uint8_t* keep_out, int32_t* count_out) {
    std::vector<uint8_t> keep(V);
    int n = prune(lp, keep.data());
    if (keep_out) std::memcpy(keep_out, keep.data(), V);
    if (count_out) *count_out = n;

    std::map<int, Mass> next;  // keyed by trie node == by token sequence
    for (const auto& entry : beam) {
      int node = entry.first;
      const Mass& m = entry.second;
      double tot = total(m);
      int last = nodes[node].token;  // -1 for the empty prefix
      if (keep[blank]) {
        Mass& s = next[node];
        s.pb = combine(s.pb, tot + (double)lp[blank]);
      }
      if (last >= 0 && keep[last]) {
        Mass& s = next[node];
        s.pnb = combine(s.pnb, m.pnb + (double)lp[last]);
      }
      for (int c = 0; c < V; ++c) {
        if (c == blank || !keep[c]) continue;
        // a repeated token starts a new symbol only after a blank
        double from = (c == last) ? m.pb : tot;
        Mass& s = next[child_of(node, c)];
        s.pnb = combine(s.pnb, from + (double)lp[c]);
      }
    }

    struct Cand {
      int node;
      Mass m;
      double tot;
    };
    std::vector<Cand> cands;
    for (const auto& kv : next) {
      double t = total(kv.second);
      if (t == NEG_INF) continue;
      cands.push_back(Cand{kv.first, kv.second, t});
    }
    std::sort(cands.begin(), cands.end(), [this](const Cand& a, const Cand& b) {
      if (a.tot != b.tot) return a.tot > b.tot;
      if (nodes[a.node].depth != nodes[b.node].depth)
        return nodes[a.node].depth < nodes[b.node].depth;
      return sequence(a.node) < sequence(b.node);
    });
    if ((int)cands.size() > K) cands.resize(K);
    if (beam_threshold > 0.0 && !cands.empty()) {
      const double floor = cands[0].tot - beam_threshold;
      size_t n = cands.size();
      while (n > 1 && cands[n - 1].tot < floor) --n;
      cands.resize(n);
    }
    beam.clear();
    for (const auto& c : cands) beam.emplace_back(c.node, c.m);
    ++frames_seen;
  }
};

}  // namespace

extern "C" {

// The float32 value of log R used by the prune comparison.
float oracle_log_r(float r) { return Decoder(2, 0, 1, r).log_r; }

// Survivor mask of `n_frames` consecutive frames (row stride V).
void oracle_prune(const float* lp, int64_t n_frames, int V, float r, uint8_t* keep,
                  int32_t* counts) {
  Decoder d(V, 0, 1, r);
  for (int64_t t = 0; t < n_frames; ++t) counts[t] = d.prune(lp + t * V, keep + t * V);
}

void* oracle_stream_create(int V, int blank, int K, float r) { return new Decoder(V, blank, K, r); }
// The optional knobs of Algorithm 1 (see the header of this file); call before feeding.
void oracle_stream_options(void* h, int top_n, double beam_threshold) {
  ((Decoder*)h)->top_n = top_n;
  ((Decoder*)h)->beam_threshold = beam_threshold;
}
void oracle_stream_merge_max(void* h, int merge_max) { ((Decoder*)h)->merge_max = merge_max != 0; }
// Survivor mask with the top-N cap.
void oracle_prune_topn(const float* lp, int64_t n_frames, int V, float r, int top_n, uint8_t* keep,
                       int32_t* counts) {
  Decoder d(V, 0, 1, r);
  d.top_n = top_n;
  for (int64_t t = 0; t < n_frames; ++t) counts[t] = d.prune(lp + t * V, keep + t * V);
}
void oracle_stream_destroy(void* h) { delete (Decoder*)h; }
void oracle_stream_reset(void* h) { ((Decoder*)h)->reset(); }

// Consume n_frames rows (stride V).  keep/counts may be null.
void oracle_stream_feed(void* h, const float* lp, int64_t n_frames, uint8_t* keep,
                        int32_t* counts) {
  Decoder* d = (Decoder*)h;
  for (int64_t t = 0; t < n_frames; ++t)
    d->step(lp + t * d->V, keep ? keep + t * d->V : nullptr, counts ? counts + t : nullptr);
}

// Current beam, best first.  tokens is [K, max_len] (sequences longer than
// max_len are truncated, lens reports the true length).  Returns the number
// of hypotheses.
int oracle_stream_results(void* h, int32_t* tokens, int32_t* lens, double* scores,
                          double* pb, double* pnb, int max_len) {
  Decoder* d = (Decoder*)h;
  int n = (int)d->beam.size();
  for (int k = 0; k < d->K; ++k) {
    if (lens) lens[k] = 0;
    if (scores) scores[k] = NEG_INF;
    if (pb) pb[k] = NEG_INF;
    if (pnb) pnb[k] = NEG_INF;
  }
  for (int k = 0; k < n; ++k) {
    std::vector<int> s = d->sequence(d->beam[k].first);
    if (lens) lens[k] = (int)s.size();
    if (tokens)
      for (int i = 0; i < (int)s.size() && i < max_len; ++i) tokens[(int64_t)k * max_len + i] = s[i];
    if (scores) scores[k] = d->total(d->beam[k].second);
    if (pb) pb[k] = d->beam[k].second.pb;
    if (pnb) pnb[k] = d->beam[k].second.pnb;
  }
  return n;
}

// Whole-batch decode.  lp is [B, T, V] with element strides (stride_b,
// stride_t); frames t >= lengths[b] are never read.  Outputs: tokens
// [B,K,max_len], lens [B,K], scores [B,K] (float64), nhyp [B]; optional
// keep [B,T,V] and counts [B,T] (entries of unread frames are left untouched).
void oracle_decode_opt(const float* lp, int64_t stride_b, int64_t stride_t, const int32_t* lengths,
                       int B, int T, int V, int blank, int K, float r, int top_n,
                       double beam_threshold, int max_len, int32_t* tokens, int32_t* lens,
                       double* scores, int32_t* nhyp, uint8_t* keep, int32_t* counts,
                       int merge_max) {
  for (int b = 0; b < B; ++b) {
    Decoder d(V, blank, K, r);
    d.top_n = top_n;
    d.beam_threshold = beam_threshold;
    d.merge_max = merge_max != 0;
    int len = lengths[b];
    if (len < 0 || len > T) {
      nhyp[b] = 0;
      for (int k = 0; k < K; ++k) {
        lens[(int64_t)b * K + k] = 0;
        scores[(int64_t)b * K + k] = NEG_INF;
      }
      continue;
    }
    for (int t = 0; t < len; ++t)
      d.step(lp + b * stride_b + t * stride_t,
             keep ? keep + ((int64_t)b * T + t) * V : nullptr,
             counts ? counts + (int64_t)b * T + t : nullptr);
    nhyp[b] = oracle_stream_results(&d, tokens + (int64_t)b * K * max_len, lens + (int64_t)b * K,
                                    scores + (int64_t)b * K, nullptr, nullptr, max_len);
  }
}

void oracle_decode(const float* lp, int64_t stride_b, int64_t stride_t, const int32_t* lengths,
                   int B, int T, int V, int blank, int K, float r, int max_len, int32_t* tokens,
                   int32_t* lens, double* scores, int32_t* nhyp, uint8_t* keep, int32_t* counts) {
  oracle_decode_opt(lp, stride_b, stride_t, lengths, B, T, V, blank, K, r, 0, 0.0, max_len, tokens,
                    lens, scores, nhyp, keep, counts, 0);
}

}  // extern "C"
