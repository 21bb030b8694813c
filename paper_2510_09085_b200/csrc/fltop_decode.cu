// Beam extension, prefix merge, top-K selection and prefix-trie maintenance
// for frame-pruned CTC prefix beam search (Algorithm 1: the loops over the
// beam and over the surviving tokens, B'.add, SelectTopK, and
// GetHighestScorePrefix after the last frame).
//
// One thread block decodes one utterance and walks its frames serially; the
// beam lives in shared memory for the whole utterance.  The frame loop is a
// chain of dependent steps, so the design minimises block barriers per frame
// (five on the common path) rather than bytes moved:
//   P1  every beam entry q gets its "stay" candidate (pb' = tot + lp[blank],
//       pnb' = pnb + lp[last(q)], plus - the prefix merge - the mass of its
//       parent extended by last(q) when the parent is in the beam); every
//       (beam entry, non-blank survivor) pair gets an extension candidate
//       unless that prefix is already in the beam.  Each candidate adds one
//       to a 512-bin histogram of its score (1/8 nat per bin).
//   P2  warp 0 scans the histogram: the bin holding the K-th best score is
//       the cut; bins above it become slot counters.  Meanwhile the other
//       warps publish last frame's trie changes and stage the next frame's
//       log-probabilities.
//   P3  candidates above the cut take their beam slot with one shared-memory
//       atomic and are written to the next beam; candidates inside the cut
//       bin are ranked exactly among themselves (a handful).
//   P5  selected extensions get their trie node by lookup-or-create, so that
//       one node id always means one token sequence; parent slots and the
//       in-beam child bits of the next frame are set.
// If the cut bin is crowded (many near-equal scores) an exact radix select
// over order-preserving integer keys replaces P3.
// Scores are float32 relative to the best total of the previous frame; the
// sum of the subtracted maxima is kept in float64.
#include "fltop_internal.h"

namespace fltop {
namespace {

constexpr int kMaxThreads = 1024;
constexpr int kCache = 4;          // candidate keys cached in registers per thread
constexpr int kFastBins = 512;     // score histogram of the fast select
constexpr float kBinsPerNat = 8.f;
constexpr int kListCap = 64;       // candidates of the cut bin ranked pairwise
constexpr int kRadixBits = 8;      // exact fallback select
constexpr int kBins = 1 << kRadixBits;
constexpr int kPasses = 32 / kRadixBits;

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

// log(exp(a) + exp(b)); symmetric in its arguments.
__device__ __forceinline__ float lse2(float a, float b) {
  const float hi = fmaxf(a, b), lo = fminf(a, b);
  if (lo == neg_inf()) return hi;
  return hi + log1pf(expf(lo - hi));
}

// Order-preserving map float -> uint32 (larger float = larger key).  Key 0 is
// reserved for "not a candidate"; -inf maps there too (probability 0 is
// dropped, as SelectTopK never keeps it).
__device__ __forceinline__ unsigned score_key(float s) {
  if (s == neg_inf()) return 0u;
  const unsigned u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_score(unsigned k) {
  const unsigned u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
  return __uint_as_float(u);
}
// Histogram bin of a candidate: monotone in the score, bin 0 holds the best.
__device__ __forceinline__ int score_bin(unsigned key) {
  const int b = __float2int_rz(-key_score(key) * kBinsPerNat);
  return min(kFastBins - 1, max(0, b));
}
// Bins are stored transposed so that the lane of warp 0 that owns bins
// [16 l, 16 l + 16) reads them without bank conflicts.
__device__ __forceinline__ int bin_addr(int bin) { return ((bin & 15) << 5) | (bin >> 4); }

__device__ __forceinline__ void cp_async8(void* smem_dst, const void* gmem_src) {
  const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(d), "l"(gmem_src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n"); }
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");
}
__device__ __forceinline__ void cp_async_wait_but_one() {
  asm volatile("cp.async.wait_group 1;\n" ::: "memory");
}

// Beam fields, each a [K] array of 32-bit words, two copies (current / next).
enum { F_NODE, F_LAST, F_PAR, F_PARNODE, F_PB, F_PNB, F_FIRST, F_LEN, F_TOT, NF };
//   NODE     trie node id of the prefix
//   LAST     its last token (-1 for the empty prefix)
//   PAR      beam slot of the prefix without its last token, -1 if not in the beam
//   PARNODE  trie node id of that parent (-1 for the empty prefix)
//   PB, PNB  log-mass ending in blank / in the last token (relative)
//   FIRST    head of the node's child list as of the start of the frame
//   LEN      number of tokens
//   TOT      lse(PB, PNB)

enum {
  SC_NBEAM_NEXT = 0, SC_MAXKEY, SC_THR, SC_LEFT, SC_CUT_COUNT, SC_CUT_BASE, SC_LISTN,
  SC_REVIVED, SC_STATUS, SC_CREATED, SC_BLANK_J0, SC_BLANK_J1,
  // exact fallback select
  SC_PREFIX, SC_SHIFT, SC_NEED, SC_TAKEALL, SC_DONE, SC_COUNT
};

// Byte offsets of the shared-memory arrays.
struct Lay {
  unsigned filt, sv, warp_sums, beam, newhead, st_pb, st_pnb, st_key, old2new, from, isext,
      dirty, inbeam, lpv, hist, rhist, list_key, list_idx, scal, total;
};

__host__ __device__ inline Lay make_layout(int K, int V) {
  Lay l;
  unsigned off = 0;
  const unsigned W = (unsigned)(V + 31) / 32;
  auto take = [&](unsigned bytes) {
    const unsigned at = off;
    off += (bytes + 7u) & ~7u;
    return at;
  };
  l.filt = take(2u * K * 8);
  l.sv = take(4u * V * 8);
  l.warp_sums = take(34 * 8);
  l.beam = take(2u * NF * K * 4);
  l.newhead = take(K * 4);
  l.st_pb = take(K * 4);
  l.st_pnb = take(K * 4);
  l.st_key = take(K * 4);
  l.old2new = take(K * 4);
  l.from = take(K * 4);
  l.isext = take(K * 4);
  l.dirty = take(K * 4);
  l.inbeam = take(2u * K * W * 4);
  l.lpv = take(2u * V * 4);
  l.hist = take(kFastBins * 4);
  l.rhist = take(kPasses * kBins * 4);
  l.list_key = take(kListCap * 4);
  l.list_idx = take(kListCap * 4);
  l.scal = take(SC_COUNT * 4);
  l.total = (off + 15u) & ~15u;
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
    const unsigned long long up = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += up;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    unsigned long long w = lane < n_warps ? warp_sums[lane] : 0ull;
    unsigned long long winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long up = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += up;
    }
    warp_sums[lane] = winc - w;  // exclusive prefix of each warp
    if (lane == 31) warp_sums[32] = winc;
  }
  __syncthreads();
  *total = warp_sums[32];
  return warp_sums[warp] + inc - v;
}

// Fast select, P2: warp 0 turns the score histogram into slot counters.
// Afterwards hist[bin] holds the number of candidates in better bins, for every
// bin up to and including the cut bin.
__device__ __forceinline__ void scan_score_histogram(unsigned* hist, int* scal, int K) {
  const int lane = threadIdx.x & 31;
  unsigned cnt[16];
  unsigned c = 0;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    cnt[i] = hist[(i << 5) | lane];
    c += cnt[i];
  }
  unsigned inc = c;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned up = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += up;
  }
  const unsigned total = __shfl_sync(0xffffffffu, inc, 31);
  const bool all = (int)total <= K;
  const unsigned hit = __ballot_sync(0xffffffffu, (int)inc >= K);
  const int owner = all ? 32 : __ffs(hit) - 1;
  unsigned acc = inc - c;
  if (lane < owner) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      hist[(i << 5) | lane] = acc;
      acc += cnt[i];
    }
  } else if (lane == owner) {
    int cut = 0;
    unsigned cut_cnt = 0;
    bool found = false;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      if (!found) {
        hist[(i << 5) | lane] = acc;
        if ((int)(acc + cnt[i]) >= K) {
          found = true;
          cut = i;
          cut_cnt = cnt[i];
        } else {
          acc += cnt[i];
        }
      }
    }
    scal[SC_THR] = 16 * lane + cut;
    scal[SC_LEFT] = K - (int)acc;      // how many of the cut bin are kept
    scal[SC_CUT_COUNT] = (int)cut_cnt; // how many are in it
    scal[SC_CUT_BASE] = (int)acc;      // first slot of the cut bin
    scal[SC_NBEAM_NEXT] = K;
  }
  if (all && lane == 0) {
    scal[SC_THR] = kFastBins;  // no cut: every candidate is kept
    scal[SC_LEFT] = 0;
    scal[SC_CUT_COUNT] = 0;
    scal[SC_CUT_BASE] = 0;
    scal[SC_NBEAM_NEXT] = (int)total;
  }
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
    const unsigned up = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += up;
  }
  const unsigned total = __shfl_sync(0xffffffffu, inc, 31);
  if (pass == 0 && (int)total <= need) {
    if (lane == 0) {  // fewer candidates than beam slots: keep every candidate
      scal[SC_PREFIX] = 0; scal[SC_SHIFT] = 0; scal[SC_NEED] = 0; scal[SC_TAKEALL] = 0;
      scal[SC_DONE] = 1; scal[SC_NBEAM_NEXT] = (int)total;
    }
    return;
  }
  const unsigned hit = __ballot_sync(0xffffffffu, (int)inc >= need);
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

__global__ void __launch_bounds__(kMaxThreads) decode_kernel(DecodeParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int b = blockIdx.x, tid = threadIdx.x, NT = blockDim.x;
  const int K = p.K, V = p.V, W = (V + 31) / 32, blank = p.blank;
  const Lay L = make_layout(K, V);

  unsigned long long* const filt_base = reinterpret_cast<unsigned long long*>(smem + L.filt);
  Survivor* const sv_base = reinterpret_cast<Survivor*>(smem + L.sv);
  unsigned long long* const warp_sums = reinterpret_cast<unsigned long long*>(smem + L.warp_sums);
  int* const beam_base = reinterpret_cast<int*>(smem + L.beam);
  int* const newhead = reinterpret_cast<int*>(smem + L.newhead);
  float* const st_pb = reinterpret_cast<float*>(smem + L.st_pb);
  float* const st_pnb = reinterpret_cast<float*>(smem + L.st_pnb);
  unsigned* const st_key = reinterpret_cast<unsigned*>(smem + L.st_key);
  int* const old2new = reinterpret_cast<int*>(smem + L.old2new);
  int* const from = reinterpret_cast<int*>(smem + L.from);
  int* const isext = reinterpret_cast<int*>(smem + L.isext);
  int* const dirty = reinterpret_cast<int*>(smem + L.dirty);
  unsigned* const inbeam_base = reinterpret_cast<unsigned*>(smem + L.inbeam);
  float* const lpv_base = reinterpret_cast<float*>(smem + L.lpv);
  unsigned* const hist = reinterpret_cast<unsigned*>(smem + L.hist);
  unsigned* const rhist = reinterpret_cast<unsigned*>(smem + L.rhist);
  unsigned* const list_key = reinterpret_cast<unsigned*>(smem + L.list_key);
  int* const list_idx = reinterpret_cast<int*>(smem + L.list_idx);
  int* const scal = reinterpret_cast<int*>(smem + L.scal);

  auto bi = [&](int buf, int f) -> int* { return beam_base + (buf * NF + f) * K; };
  auto bf = [&](int buf, int f) -> float* { return reinterpret_cast<float*>(bi(buf, f)); };
  auto filt = [&](int buf) -> unsigned long long* { return filt_base + buf * K; };
  auto svbuf = [&](int t) -> Survivor* { return sv_base + (t & 3) * V; };
  auto lpvbuf = [&](int t) -> float* { return lpv_base + (t & 1) * V; };
  auto ibbuf = [&](int t) -> unsigned* { return inbeam_base + (t & 1) * K * W; };

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
  for (int i = tid; i < 2 * K * W; i += NT) inbeam_base[i] = 0u;
  for (int i = tid; i < 2 * V; i += NT) lpv_base[i] = neg_inf();
  for (int i = tid; i < kFastBins; i += NT) hist[i] = 0u;
  for (int i = tid; i < K; i += NT) {
    dirty[i] = 0;
    old2new[i] = -1;
  }
  if (tid == 0) {
    scal[SC_BLANK_J0] = -1; scal[SC_BLANK_J1] = -1;
    scal[SC_REVIVED] = 0; scal[SC_STATUS] = 0; scal[SC_CREATED] = 0;
    scal[SC_MAXKEY] = 0; scal[SC_LISTN] = 0;
  }
  int created = 0, live_sum = 0;
  int cur = 0, nb, n_nodes, frames_seen;
  double offset;
  if (do_reset) {
    nb = bad_len && !p.streaming ? 0 : 1;
    n_nodes = 1;
    offset = 0.0;
    frames_seen = 0;
    if (tid == 0) {
      bi(0, F_NODE)[0] = 0; bi(0, F_LAST)[0] = -1; bi(0, F_PAR)[0] = -1; bi(0, F_PARNODE)[0] = -1;
      bf(0, F_PB)[0] = 0.f; bf(0, F_PNB)[0] = neg_inf(); bi(0, F_FIRST)[0] = -1;
      bi(0, F_LEN)[0] = 0; bf(0, F_TOT)[0] = 0.f; filt(0)[0] = 0ull;
      TrieNode root;
      root.parent = -1; root.token = -1; root.first_child = -1; root.next_sibling = -1;
      root.depth = 0; root.pad = 0; root.child_filter = 0ull;
      nodes[0] = root;
    }
  } else {
    const StateHeader* hd = reinterpret_cast<const StateHeader*>(st);
    nb = hd->nbeam; n_nodes = hd->n_nodes; frames_seen = hd->frames; offset = hd->offset;
    status |= hd->status;
    const int32_t* a = st + kStateHeaderWords;
    for (int i = tid; i < nb; i += NT) {
      bi(0, F_NODE)[i] = a[i]; bi(0, F_LAST)[i] = a[K + i]; bi(0, F_PAR)[i] = a[2 * K + i];
      bi(0, F_PARNODE)[i] = a[3 * K + i];
      const float pb = __int_as_float(a[4 * K + i]), pnb = __int_as_float(a[5 * K + i]);
      bf(0, F_PB)[i] = pb; bf(0, F_PNB)[i] = pnb; bf(0, F_TOT)[i] = __int_as_float(a[10 * K + i]);
      bi(0, F_FIRST)[i] = a[6 * K + i]; bi(0, F_LEN)[i] = a[7 * K + i];
      filt(0)[i] = reinterpret_cast<const unsigned long long*>(a + 8 * K)[i];
    }
  }

  // ---- prologue: survivors of frames 0 and 1, log-prob table of frame 0 --------------
  const int32_t* counts = p.counts + (int64_t)b * p.T;
  const Survivor* entries = p.entries + (int64_t)b * p.T * V;
  int c0 = len > 0 ? counts[0] : 0;
  int c1 = len > 1 ? counts[1] : 0;
  int c2 = len > 2 ? counts[2] : 0;
  for (int j = tid; j < c0; j += NT) cp_async8(&svbuf(0)[j], &entries[j]);
  cp_async_commit();
  for (int j = tid; j < c1; j += NT) cp_async8(&svbuf(1)[j], &entries[(int64_t)V + j]);
  cp_async_commit();
  cp_async_wait_all();
  __syncthreads();
  for (int j = tid; j < c0; j += NT) {
    const Survivor s = svbuf(0)[j];
    lpvbuf(0)[s.token] = s.logp;
    if (s.token == blank) scal[SC_BLANK_J0] = j;
  }
  // in-beam child bits of a beam carried over from the previous chunk
  for (int i = tid; i < nb; i += NT) {
    const int par = bi(0, F_PAR)[i];
    if (par >= 0) {
      const int e = bi(0, F_LAST)[i];
      atomicOr(&ibbuf(0)[par * W + (e >> 5)], 1u << (e & 31));
    }
  }
  int nb_prev = 0;  // size of the beam whose trie changes are still unpublished
  __syncthreads();

  for (int t = 0; t < len; ++t) {
    const int nxt = cur ^ 1;
    const int Scur = c0;
    const Survivor* const sv = svbuf(t);
    const float* const lpv = lpvbuf(t);
    const unsigned* const ib = ibbuf(t);
    int* const c_last = bi(cur, F_LAST);
    int* const c_par = bi(cur, F_PAR);
    float* const c_pb = bf(cur, F_PB);
    float* const c_pnb = bf(cur, F_PNB);
    float* const c_tot = bf(cur, F_TOT);

    // survivors of frame t+2 start their way to shared memory; count of frame t+3
    if (t + 2 < len) {
      const Survivor* src = entries + (int64_t)(t + 2) * V;
      Survivor* dst = svbuf(t + 2);
      for (int j = tid; j < c2; j += NT) cp_async8(&dst[j], &src[j]);
    }
    cp_async_commit();
    const int c3 = (t + 3 < len) ? counts[t + 3] : 0;

    const int blank_j = scal[SC_BLANK_J0 + (t & 1)];
    const int Snb = Scur - (blank_j >= 0 ? 1 : 0);
    const int ncand = nb + nb * Snb;

    auto ext_key = [&](int idx) -> unsigned {
      const int e = idx - nb;
      const int q = e / Snb;
      int j = e - q * Snb;
      if (blank_j >= 0 && j >= blank_j) ++j;
      const Survivor s = sv[j];
      if ((ib[q * W + (s.token >> 5)] >> (s.token & 31)) & 1u) return 0u;  // merged into a stay
      const float base = (s.token == c_last[q]) ? c_pb[q] : c_tot[q];
      return score_key(base + s.logp);
    };
    auto stay_key = [&](int i) -> unsigned {
      const int e = c_last[i];
      const float npb = c_tot[i] + lpv[blank];
      float npnb = neg_inf();
      if (e >= 0) {
        const float le = lpv[e];
        npnb = c_pnb[i] + le;
        const int par = c_par[i];
        if (par >= 0) {
          const float base = (c_last[par] == e) ? c_pb[par] : c_tot[par];
          npnb = lse2(npnb, base + le);
        }
      }
      st_pb[i] = npb;
      st_pnb[i] = npnb;
      const unsigned key = score_key(lse2(npb, npnb));
      st_key[i] = key;
      return key;
    };
    auto cand_key = [&](int idx) -> unsigned { return idx < nb ? st_key[idx] : ext_key(idx); };

    // ---- P1: evaluate every candidate once, score histogram, running maximum ----------
    unsigned kc[kCache];
    {
      unsigned local_max = 0u;
#pragma unroll
      for (int k = 0; k < kCache; ++k) {
        const int idx = tid + k * NT;
        unsigned key = 0u;
        if (idx < ncand) key = idx < nb ? stay_key(idx) : ext_key(idx);
        kc[k] = key;
        if (key) atomicAdd(&hist[bin_addr(score_bin(key))], 1u);
        local_max = max(local_max, key);
      }
      for (int idx = tid + kCache * NT; idx < ncand; idx += NT) {
        const unsigned key = idx < nb ? stay_key(idx) : ext_key(idx);
        if (key) atomicAdd(&hist[bin_addr(score_bin(key))], 1u);
        local_max = max(local_max, key);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1)
        local_max = max(local_max, __shfl_xor_sync(0xffffffffu, local_max, o));
      if ((tid & 31) == 0 && local_max)
        atomicMax(reinterpret_cast<unsigned*>(&scal[SC_MAXKEY]), local_max);
      if (tid == 0) scal[SC_BLANK_J0 + ((t + 1) & 1)] = -1;
    }
    cp_async_wait_but_one();  // survivors of frame t+1 have landed (this thread's part)
    __syncthreads();          // B1

    // ---- P2: warp 0 finds the cut; the others do the bookkeeping ------------------------
    if (tid < 32) {
      scan_score_histogram(hist, scal, K);
    } else {
      // publish the child lists changed last frame: to HBM and to the surviving entry
      const int o = cur ^ 1;  // last frame's beam
      const int n_pub = max(nb_prev, nb);
      if (tid == 32) scal[SC_REVIVED] = 0;
      for (int i = tid - 32; i < n_pub; i += NT - 32) {
        if (i < nb_prev && dirty[i]) {
          dirty[i] = 0;
          const int head = newhead[i];
          const unsigned long long f = filt(o)[i];
          TrieNode* n = &nodes[bi(o, F_NODE)[i]];
          n->first_child = head;
          n->child_filter = f;
          const int s = old2new[i];
          if (s >= 0) {
            bi(cur, F_FIRST)[s] = head;
            filt(cur)[s] = f;
          }
        }
        old2new[i] = -1;  // from here on: slot of current entry i in the next beam
      }
      // log-prob table: forget frame t, stage frame t+1
      float* lp_now = lpvbuf(t);
      for (int j = tid - 32; j < Scur; j += NT - 32) lp_now[sv[j].token] = neg_inf();
      if (t + 1 < len) {
        float* lp_next = lpvbuf(t + 1);
        const Survivor* sn = svbuf(t + 1);
        for (int j = tid - 32; j < c1; j += NT - 32) {
          const Survivor s = sn[j];
          lp_next[s.token] = s.logp;
          if (s.token == blank) scal[SC_BLANK_J0 + ((t + 1) & 1)] = j;
        }
      }
    }
    __syncthreads();  // B2

    // ---- P3: selected candidates take their slots in the next beam ---------------------
    const int thr = scal[SC_THR], left = scal[SC_LEFT];
    const int cut_count = scal[SC_CUT_COUNT], cut_base = scal[SC_CUT_BASE];
    const unsigned maxkey = (unsigned)scal[SC_MAXKEY];
    const int nbn = maxkey ? scal[SC_NBEAM_NEXT] : 0;
    const float best = maxkey ? key_score(maxkey) : 0.f;
    const bool take_all = cut_count == left;  // also true when there is no cut at all
    const bool use_list = !take_all && cut_count <= kListCap;

    auto place = [&](int idx, unsigned key, int slot) {
      if (idx < nb) {
        old2new[idx] = slot;
        bi(nxt, F_NODE)[slot] = bi(cur, F_NODE)[idx];
        bi(nxt, F_LAST)[slot] = c_last[idx];
        bi(nxt, F_PARNODE)[slot] = bi(cur, F_PARNODE)[idx];
        bf(nxt, F_PB)[slot] = st_pb[idx] - best;
        bf(nxt, F_PNB)[slot] = st_pnb[idx] - best;
        bf(nxt, F_TOT)[slot] = key_score(key) - best;
        bi(nxt, F_FIRST)[slot] = bi(cur, F_FIRST)[idx];
        bi(nxt, F_LEN)[slot] = bi(cur, F_LEN)[idx];
        filt(nxt)[slot] = filt(cur)[idx];
        from[slot] = idx;
        isext[slot] = 0;
      } else {
        const int e = idx - nb;
        const int q = e / Snb;
        int j = e - q * Snb;
        if (blank_j >= 0 && j >= blank_j) ++j;
        const float sc = key_score(key) - best;
        bi(nxt, F_NODE)[slot] = -1;
        bi(nxt, F_LAST)[slot] = sv[j].token;
        bi(nxt, F_PARNODE)[slot] = bi(cur, F_NODE)[q];
        bf(nxt, F_PB)[slot] = neg_inf();
        bf(nxt, F_PNB)[slot] = sc;
        bf(nxt, F_TOT)[slot] = sc;
        bi(nxt, F_FIRST)[slot] = -1;
        bi(nxt, F_LEN)[slot] = bi(cur, F_LEN)[q] + 1;
        filt(nxt)[slot] = 0ull;
        from[slot] = q;
        isext[slot] = 1;
      }
    };

    for (int i = tid; i < nb; i += NT) newhead[i] = bi(cur, F_FIRST)[i];

    if (take_all || use_list) {
      auto assign = [&](int idx, unsigned key) {
        if (!key) return;
        const int bin = score_bin(key);
        if (bin < thr || (bin == thr && take_all)) {
          place(idx, key, (int)atomicAdd(&hist[bin_addr(bin)], 1u));
        } else if (bin == thr) {
          const int li = atomicAdd(&scal[SC_LISTN], 1);
          list_key[li] = key;
          list_idx[li] = idx;
        }
      };
#pragma unroll
      for (int k = 0; k < kCache; ++k) {
        const int idx = tid + k * NT;
        if (idx < ncand) assign(idx, kc[k]);
      }
      for (int idx = tid + kCache * NT; idx < ncand; idx += NT) assign(idx, cand_key(idx));
      if (!take_all) {
        __syncthreads();  // B3: the cut bin's members are listed
        // exact order inside the cut bin: score, then candidate index
        for (int li = tid; li < cut_count; li += NT) {
          const unsigned key = list_key[li];
          const int idx = list_idx[li];
          int rank = 0;
          for (int j = 0; j < cut_count; ++j) {
            const unsigned kj = list_key[j];
            rank += (kj > key || (kj == key && list_idx[j] < idx)) ? 1 : 0;
          }
          if (rank < left) place(idx, key, cut_base + rank);
        }
      }
    } else {
      // ---- exact fallback: radix select over the integer keys ------------------------
      for (int i = tid; i < kPasses * kBins; i += NT) rhist[i] = 0u;
      if (tid == 0) {
        scal[SC_PREFIX] = 0; scal[SC_NEED] = K; scal[SC_DONE] = 0; scal[SC_TAKEALL] = 0;
        scal[SC_SHIFT] = 0;
      }
      __syncthreads();
      for (int pass = 0; pass < kPasses; ++pass) {
        const int sh = 32 - kRadixBits * (pass + 1);
        const unsigned prefix = (unsigned)scal[SC_PREFIX];
        unsigned* h = rhist + pass * kBins;
        for (int idx = tid; idx < ncand; idx += NT) {
          const unsigned key = cand_key(idx);
          if (key && (pass == 0 || (key >> (sh + kRadixBits)) == prefix))
            atomicAdd(&h[(key >> sh) & (kBins - 1)], 1u);
        }
        __syncthreads();
        if (tid < 32) resolve_digit(h, scal, pass, sh);
        __syncthreads();
        if (scal[SC_DONE]) break;  // block-uniform
      }
      const int sh = scal[SC_SHIFT];
      const unsigned prefix = (unsigned)scal[SC_PREFIX];
      const int need = scal[SC_NEED];
      const bool r_all = scal[SC_TAKEALL] != 0;
      unsigned long long mine = 0ull;
      for (int idx = tid; idx < ncand; idx += NT) {
        const unsigned key = cand_key(idx);
        if (key) {
          const unsigned hk = key >> sh;
          mine += (hk > prefix) ? 1ull : ((hk == prefix) ? (1ull << 32) : 0ull);
        }
      }
      unsigned long long total;
      const unsigned long long excl = block_exclusive_scan(mine, warp_sums, &total);
      int gt_rank = (int)(excl & 0xffffffffull), eq_rank = (int)(excl >> 32);
      const int total_gt = (int)(total & 0xffffffffull);
      for (int idx = tid; idx < ncand; idx += NT) {
        const unsigned key = cand_key(idx);
        if (!key) continue;
        const unsigned hk = key >> sh;
        if (hk > prefix) {
          place(idx, key, gt_rank++);
        } else if (hk == prefix) {
          if (r_all || eq_rank < need) place(idx, key, total_gt + eq_rank);
          ++eq_rank;
        }
      }
    }
    __syncthreads();  // B4: the next beam is complete except for node ids and parent slots

    // ---- P5: trie nodes, parent slots, in-beam child bits of the next frame ------------
    unsigned* const ib_next = ibbuf(t + 1);
    for (int s = tid; s < nbn; s += NT) {
      const int q = from[s];
      const int tok = bi(nxt, F_LAST)[s];
      int par;
      if (isext[s]) {
        par = old2new[q];
        int node = -1;
        if ((filt(cur)[q] >> (tok & 63)) & 1ull) {
          // a child with this filter bit exists: walk the parent's child list
          int id = bi(cur, F_FIRST)[q];
          for (int it = 0; id >= 0 && it <= V; ++it) {
            const int4 rec = *reinterpret_cast<const int4*>(&nodes[id]);  // parent, token, first, next
            if (rec.y == tok) {
              node = id;
              bi(nxt, F_FIRST)[s] = rec.z;
              filt(nxt)[s] = nodes[id].child_filter;
              scal[SC_REVIVED] = 1;
              break;
            }
            id = rec.w;
          }
        }
        if (node < 0) {
          const int id = n_nodes + s;
          if (id < p.nodes_per_utt) {
            const int prev = atomicExch(&newhead[q], id);
            atomicOr(&filt(cur)[q], 1ull << (tok & 63));
            dirty[q] = 1;
            TrieNode n;
            n.parent = bi(cur, F_NODE)[q]; n.token = tok; n.first_child = -1;
            n.next_sibling = prev; n.depth = bi(nxt, F_LEN)[s]; n.pad = 0; n.child_filter = 0ull;
            nodes[id] = n;
            node = id;
            ++created;
          } else {
            node = 0;
            scal[SC_STATUS] = 2;  // FLTOP_ST_ARENA_FULL
          }
        }
        bi(nxt, F_NODE)[s] = node;
      } else {
        const int op = c_par[q];
        par = op >= 0 ? old2new[op] : -1;
      }
      bi(nxt, F_PAR)[s] = par;
      if (par >= 0) atomicOr(&ib_next[par * W + (tok >> 5)], 1u << (tok & 31));
    }
    {
      unsigned* const ib_now = ibbuf(t);
      for (int i = tid; i < nb; i += NT) {
        const int par = c_par[i];
        if (par >= 0) ib_now[par * W + (c_last[i] >> 5)] = 0u;
      }
    }
    for (int i = tid; i < kFastBins; i += NT) hist[i] = 0u;
    if (tid == 0) {
      scal[SC_MAXKEY] = 0;
      scal[SC_LISTN] = 0;
    }
    if (!maxkey) status |= 8;  // FLTOP_ST_EMPTY_BEAM
    offset += (double)best;
    __syncthreads();  // B5

    if (scal[SC_REVIVED]) {
      // a prefix came back into the beam: entries that extend it find their parent again
      for (int s = tid; s < nbn; s += NT) {
        if (isext[s] && bi(nxt, F_NODE)[s] < n_nodes) {
          const int x = bi(nxt, F_NODE)[s];
          for (int s2 = 0; s2 < nbn; ++s2) {
            if (bi(nxt, F_PARNODE)[s2] == x && bi(nxt, F_PAR)[s2] != s) {
              bi(nxt, F_PAR)[s2] = s;
              const int tk = bi(nxt, F_LAST)[s2];
              atomicOr(&ib_next[s * W + (tk >> 5)], 1u << (tk & 31));
            }
          }
        }
      }
      __syncthreads();
    }
    n_nodes += nbn;
    live_sum += nbn;
    nb_prev = nb;
    nb = nbn;
    cur = nxt;
    c0 = c1; c1 = c2; c2 = c3;
  }
  frames_seen += len;

  // trie changes of the last frame
  for (int i = tid; i < nb_prev; i += NT) {
    if (dirty[i]) {
      dirty[i] = 0;
      const int o = cur ^ 1;
      const int head = newhead[i];
      const unsigned long long f = filt(o)[i];
      TrieNode* n = &nodes[bi(o, F_NODE)[i]];
      n->first_child = head;
      n->child_filter = f;
      const int s = old2new[i];
      if (s >= 0) {
        bi(cur, F_FIRST)[s] = head;
        filt(cur)[s] = f;
      }
    }
  }
  __syncthreads();
  status |= scal[SC_STATUS];
  if (p.stats) {
    if (created) atomicAdd(&scal[SC_CREATED], created);
    __syncthreads();
    if (tid == 0) {
      int32_t* o = p.stats + 4 * (int64_t)b;
      o[0] = len; o[1] = scal[SC_CREATED]; o[2] = live_sum; o[3] = n_nodes;
    }
  }

  // ---- keep the beam for the next chunk (streaming) -----------------------------------
  if (p.streaming) {
    int32_t* a = st + kStateHeaderWords;
    for (int i = tid; i < nb; i += NT) {
      a[i] = bi(cur, F_NODE)[i]; a[K + i] = bi(cur, F_LAST)[i]; a[2 * K + i] = bi(cur, F_PAR)[i];
      a[3 * K + i] = bi(cur, F_PARNODE)[i];
      a[4 * K + i] = bi(cur, F_PB)[i]; a[5 * K + i] = bi(cur, F_PNB)[i];
      a[6 * K + i] = bi(cur, F_FIRST)[i]; a[7 * K + i] = bi(cur, F_LEN)[i];
      reinterpret_cast<unsigned long long*>(a + 8 * K)[i] = filt(cur)[i];
      a[10 * K + i] = bi(cur, F_TOT)[i];
    }
    if (tid == 0) {
      StateHeader* hd = reinterpret_cast<StateHeader*>(st);
      hd->nbeam = nb; hd->n_nodes = n_nodes; hd->frames = frames_seen;
      hd->status = status & ~1;  // a bad chunk length is not sticky
      hd->offset = offset;
    }
  }

  // ---- hypotheses, best first (GetHighestScorePrefix over the whole beam) ----------
  if (do_emit) {
    const int Lout = p.L;
    const float* tot = bf(cur, F_TOT);
    bool truncated = false;
    for (int i = tid; i < nb; i += NT) {
      const float ti = tot[i];
      int rank = 0;
      for (int j = 0; j < nb; ++j) {
        const float tj = tot[j];
        rank += (tj > ti || (tj == ti && j < i)) ? 1 : 0;
      }
      const int64_t o = (int64_t)b * K + rank;
      p.out_scores[o] = (float)(offset + (double)ti);
      const int n = bi(cur, F_LEN)[i];
      p.out_lens[o] = n;
      if (n > Lout) truncated = true;
      int32_t* dst = p.out_tokens + o * Lout;
      int node = bi(cur, F_NODE)[i];
      for (int d = n - 1; d >= 0 && node > 0; --d) {
        const int2 rec = *reinterpret_cast<const int2*>(&nodes[node]);  // parent, token
        if (d < Lout) dst[d] = rec.y;
        node = rec.x;
      }
    }
    for (int k = nb + tid; k < K; k += NT) {
      p.out_lens[(int64_t)b * K + k] = 0;
      p.out_scores[(int64_t)b * K + k] = neg_inf();
    }
    if (truncated) atomicOr(&scal[SC_STATUS], 4);  // FLTOP_ST_TRUNCATED
    __syncthreads();
    status |= scal[SC_STATUS];
    if (tid == 0) p.out_nhyp[b] = nb;
  }
  if (tid == 0 && p.out_status) p.out_status[b] = status;
}

}  // namespace

size_t decode_smem_bytes(int K, int V) { return make_layout(K, V).total; }

int decode_block_threads(int K, int V) {
  // about four candidates per thread when every token survives, at most 1024
  long long want = ((long long)K * (V < 32 ? V : 32) + 3) / 4;
  if (want < K) want = K;
  int nt = (int)((want + 31) / 32 * 32);
  if (nt < 64) nt = 64;
  if (nt > kMaxThreads) nt = kMaxThreads;
  return nt;
}

cudaError_t decode_prepare(int K, int V) {
  return cudaFuncSetAttribute(decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)decode_smem_bytes(K, V));
}

cudaError_t launch_decode(const DecodeParams& p, cudaStream_t s) {
  if (p.B == 0) return cudaSuccess;
  decode_kernel<<<p.B, decode_block_threads(p.K, p.V), decode_smem_bytes(p.K, p.V), s>>>(p);
  return cudaGetLastError();
}

}  // namespace fltop
