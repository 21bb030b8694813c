// Beam extension, prefix merge, top-K selection and prefix-trie maintenance
// for frame-pruned CTC prefix beam search (Algorithm 1: the loops over the
// beam and over the surviving tokens, B'.add, SelectTopK, and
// GetHighestScorePrefix after the last frame).
//
// One thread block decodes one utterance and walks its frames serially; the
// beam lives in shared memory for the whole utterance.  Per frame:
//   1. the frame's survivor list (written by the prune kernel) is already in
//      shared memory, prefetched with cp.async during the previous frame;
//   2. every beam entry q gets its "stay" candidate: pb' = tot + lp[blank],
//      pnb' = pnb + lp[last(q)], plus - this is the prefix merge - the mass of
//      its parent extended by last(q) when the parent is in the beam;
//   3. every (beam entry, non-blank survivor) pair gets an extension candidate
//      unless that extension names a prefix already in the beam (step 2 took
//      its mass);
//   4. the K best candidates are found with a most-significant-digit radix
//      select over order-preserving integer keys (shared-memory histograms);
//   5. the selected candidates are compacted into the next beam; selected
//      extensions get their trie node by lookup-or-create so that one node id
//      always means one token sequence.
// Scores are float32 relative to the best total of the previous frame; the
// sum of the subtracted maxima is kept in float64.
#include "fltop_internal.h"

namespace fltop {
namespace {

constexpr int kMaxThreads = 1024;
constexpr int kCache = 4;        // candidate keys cached in registers per thread
constexpr int kRadixBits = 8;
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

__device__ __forceinline__ void cp_async8(void* smem_dst, const void* gmem_src) {
  const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(d), "l"(gmem_src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n"); }
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");
}

// Shared-memory carve-up.  All arrays are 4-byte words except child filters.
struct Beam {
  int* node;       // trie node id of the prefix
  int* last;       // its last token (-1 for the empty prefix)
  int* par;        // beam slot of the prefix without its last token, -1 if not in the beam
  int* parnode;    // trie node id of that parent (-1 for the empty prefix)
  float* pb;       // log-mass ending in blank, relative
  float* pnb;      // log-mass ending in last token, relative
  int* first;      // head of the node's child list
  int* len;        // number of tokens
  unsigned long long* filt;  // the node's child filter
};

struct Smem {
  Beam beam[2];
  float* tot;        // [K] lse(pb, pnb) of the current beam
  float* st_pb;      // [K] stay candidate
  float* st_pnb;     // [K]
  unsigned* st_key;  // [K]
  int* old2new;      // [K] slot of a surviving entry in the next beam, else -1
  int* from;         // [K] next-beam slot -> current slot it derives from
  int* isext;        // [K] next-beam slot is a fresh extension
  int* dirty;        // [K] child list of the current entry changed this frame
  unsigned* inbeam;  // [K * W] bit c of row q: prefix q+c is in the beam
  float* lpv;        // [V] logp of surviving tokens, -inf otherwise
  Survivor* sv[2];   // [V] survivor list, double buffered
  unsigned* hist;    // [kPasses * kBins]
  unsigned long long* warp_sums;  // [34] per-warp partial sums + block total
  int* scal;         // small scalars, see enum below
};
enum {
  SC_NBEAM_NEXT = 0, SC_MAXKEY, SC_PREFIX, SC_SHIFT, SC_NEED, SC_TAKEALL, SC_DONE, SC_REVIVED,
  SC_STATUS, SC_BLANK_J, SC_CREATED, SC_COUNT
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__host__ __device__ inline size_t smem_layout(int K, int V, unsigned char* base, Smem* s) {
  size_t off = 0;
  auto take = [&](size_t bytes, size_t align) {
    off = align_up(off, align);
    size_t at = off;
    off += bytes;
    return at;
  };
  const int W = (V + 31) / 32;
  size_t o;
#define FLTOP_TAKE(field, type, count, align) \
  o = take(sizeof(type) * (size_t)(count), align); \
  if (s) s->field = reinterpret_cast<type*>(base + o);
  for (int i = 0; i < 2; ++i) {
    FLTOP_TAKE(beam[i].filt, unsigned long long, K, 8)
    FLTOP_TAKE(beam[i].node, int, K, 4)
    FLTOP_TAKE(beam[i].last, int, K, 4)
    FLTOP_TAKE(beam[i].par, int, K, 4)
    FLTOP_TAKE(beam[i].parnode, int, K, 4)
    FLTOP_TAKE(beam[i].pb, float, K, 4)
    FLTOP_TAKE(beam[i].pnb, float, K, 4)
    FLTOP_TAKE(beam[i].first, int, K, 4)
    FLTOP_TAKE(beam[i].len, int, K, 4)
  }
  FLTOP_TAKE(sv[0], Survivor, V, 8)
  FLTOP_TAKE(sv[1], Survivor, V, 8)
  FLTOP_TAKE(warp_sums, unsigned long long, 34, 8)
  FLTOP_TAKE(tot, float, K, 4)
  FLTOP_TAKE(st_pb, float, K, 4)
  FLTOP_TAKE(st_pnb, float, K, 4)
  FLTOP_TAKE(st_key, unsigned, K, 4)
  FLTOP_TAKE(old2new, int, K, 4)
  FLTOP_TAKE(from, int, K, 4)
  FLTOP_TAKE(isext, int, K, 4)
  FLTOP_TAKE(dirty, int, K, 4)
  FLTOP_TAKE(inbeam, unsigned, (size_t)K * W, 4)
  FLTOP_TAKE(lpv, float, V, 4)
  FLTOP_TAKE(hist, unsigned, kPasses * kBins, 4)
  FLTOP_TAKE(scal, int, SC_COUNT, 4)
#undef FLTOP_TAKE
  return align_up(off, 16);
}

// Exclusive block scan of a packed pair of counters (low / high 32 bits).
// Returns the exclusive prefix of the calling thread; *total gets the block sum.
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

// After a histogram pass over digit `shift`, warp 0 finds the bin that holds
// the need-th largest key of the current prefix group.
__device__ __forceinline__ void resolve_digit(const Smem& S, int pass, int shift) {
  const int lane = threadIdx.x & 31;
  const unsigned* h = S.hist + pass * kBins;
  const int need = S.scal[SC_NEED];
  // lane l owns bins [255 - 8l - 7, 255 - 8l], walked from the top
  constexpr int PER = kBins / 32;
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
    // fewer candidates than beam slots: keep every candidate
    if (lane == 0) {
      S.scal[SC_PREFIX] = 0;
      S.scal[SC_SHIFT] = 0;
      S.scal[SC_NEED] = 0;
      S.scal[SC_TAKEALL] = 0;
      S.scal[SC_DONE] = 1;
      S.scal[SC_NBEAM_NEXT] = (int)total;
    }
    return;
  }
  const unsigned hit = __ballot_sync(0xffffffffu, (int)inc >= need);
  const int owner = __ffs(hit) - 1;  // hit != 0 because total > need >= 1 or group size >= need
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
    S.scal[SC_PREFIX] = (int)(((unsigned)S.scal[SC_PREFIX] << kRadixBits) | (unsigned)d);
    S.scal[SC_SHIFT] = shift;
    S.scal[SC_NEED] = left;
    const int all = ((int)cnt == left);
    S.scal[SC_TAKEALL] = all;
    S.scal[SC_DONE] = (all || shift == 0) ? 1 : 0;
  }
}

__global__ void __launch_bounds__(kMaxThreads) decode_kernel(DecodeParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Smem S;
  smem_layout(p.K, p.V, smem_raw, &S);
  const int b = blockIdx.x, tid = threadIdx.x, NT = blockDim.x;
  const int K = p.K, V = p.V, W = (V + 31) / 32, blank = p.blank;

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
  int32_t* st = p.streaming ? p.state + (int64_t)b * (kStateHeaderWords + kStateWordsPerSlot * (int64_t)K)
                            : nullptr;

  // ---- initialise shared state -------------------------------------------------
  for (int i = tid; i < K * W; i += NT) S.inbeam[i] = 0u;
  for (int i = tid; i < V; i += NT) S.lpv[i] = neg_inf();
  for (int i = tid; i < K; i += NT) {
    S.dirty[i] = 0;
    S.old2new[i] = -1;
  }
  if (tid == 0) {
    S.scal[SC_BLANK_J] = -1;
    S.scal[SC_REVIVED] = 0;
    S.scal[SC_STATUS] = 0;
    S.scal[SC_CREATED] = 0;
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
      Beam& B0 = S.beam[0];
      B0.node[0] = 0; B0.last[0] = -1; B0.par[0] = -1; B0.parnode[0] = -1;
      B0.pb[0] = 0.f; B0.pnb[0] = neg_inf(); B0.first[0] = -1; B0.len[0] = 0; B0.filt[0] = 0ull;
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
    Beam& B0 = S.beam[0];
    for (int i = tid; i < nb; i += NT) {
      B0.node[i] = a[i]; B0.last[i] = a[K + i]; B0.par[i] = a[2 * K + i];
      B0.parnode[i] = a[3 * K + i];
      B0.pb[i] = __int_as_float(a[4 * K + i]); B0.pnb[i] = __int_as_float(a[5 * K + i]);
      B0.first[i] = a[6 * K + i]; B0.len[i] = a[7 * K + i];
      B0.filt[i] = reinterpret_cast<const unsigned long long*>(a + 8 * K)[i];
    }
  }

  // ---- frame loop ----------------------------------------------------------------
  const int32_t* counts = p.counts + (int64_t)b * p.T;
  const Survivor* entries = p.entries + (int64_t)b * p.T * V;
  int cnt0 = len > 0 ? counts[0] : 0;
  int cnt1 = len > 1 ? counts[1] : 0;
  for (int j = tid; j < cnt0; j += NT) cp_async8(&S.sv[0][j], &entries[j]);
  cp_async_commit();
  cp_async_wait_all();
  __syncthreads();

  for (int t = 0; t < len; ++t) {
    const int buf = t & 1;
    const int Scur = cnt0;
    Beam& C = S.beam[cur];
    Beam& N = S.beam[cur ^ 1];
    // prefetch the next frame's survivors and the count of the one after
    if (t + 1 < len) {
      const Survivor* src = entries + (int64_t)(t + 1) * V;
      for (int j = tid; j < cnt1; j += NT) cp_async8(&S.sv[buf ^ 1][j], &src[j]);
    }
    cp_async_commit();
    const int cnt2 = (t + 2 < len) ? counts[t + 2] : 0;

    // P0: dense logp table, totals, in-beam child bits, histogram reset
    for (int j = tid; j < Scur; j += NT) {
      const Survivor s = S.sv[buf][j];
      S.lpv[s.token] = s.logp;
      if (s.token == blank) S.scal[SC_BLANK_J] = j;
    }
    for (int i = tid; i < nb; i += NT) {
      S.tot[i] = lse2(C.pb[i], C.pnb[i]);
      const int par = C.par[i];
      if (par >= 0) {
        const int e = C.last[i];
        atomicOr(&S.inbeam[par * W + (e >> 5)], 1u << (e & 31));
      }
    }
    for (int i = tid; i < kPasses * kBins; i += NT) S.hist[i] = 0u;
    if (tid == 0) {
      S.scal[SC_MAXKEY] = 0;
      S.scal[SC_PREFIX] = 0;
      S.scal[SC_NEED] = K;
      S.scal[SC_DONE] = 0;
      S.scal[SC_NBEAM_NEXT] = K;
      S.scal[SC_REVIVED] = 0;
    }
    __syncthreads();  // A

    const int blank_j = S.scal[SC_BLANK_J];
    const int Snb = Scur - (blank_j >= 0 ? 1 : 0);
    const int ncand = nb + nb * Snb;

    auto ext_key = [&](int idx) -> unsigned {
      const int e = idx - nb;
      const int q = e / Snb;
      int j = e - q * Snb;
      if (blank_j >= 0 && j >= blank_j) ++j;
      const Survivor s = S.sv[buf][j];
      if ((S.inbeam[q * W + (s.token >> 5)] >> (s.token & 31)) & 1u) return 0u;  // merged
      const float base = (s.token == C.last[q]) ? C.pb[q] : S.tot[q];
      return score_key(base + s.logp);
    };
    auto stay_key = [&](int i) -> unsigned {
      const int e = C.last[i];
      const float npb = S.tot[i] + S.lpv[blank];
      float npnb = neg_inf();
      if (e >= 0) {
        const float le = S.lpv[e];
        npnb = C.pnb[i] + le;
        const int par = C.par[i];
        if (par >= 0) {
          const float base = (C.last[par] == e) ? C.pb[par] : S.tot[par];
          npnb = lse2(npnb, base + le);
        }
      }
      S.st_pb[i] = npb;
      S.st_pnb[i] = npnb;
      const unsigned key = score_key(lse2(npb, npnb));
      S.st_key[i] = key;
      return key;
    };

    // P1: evaluate every candidate once, first histogram pass, running maximum
    unsigned kc[kCache];
    {
      unsigned local_max = 0u;
      unsigned* h = S.hist;
#pragma unroll
      for (int k = 0; k < kCache; ++k) {
        const int idx = tid + k * NT;
        unsigned key = 0u;
        if (idx < ncand) key = idx < nb ? stay_key(idx) : ext_key(idx);
        kc[k] = key;
        if (key) atomicAdd(&h[key >> 24], 1u);
        local_max = max(local_max, key);
      }
      for (int idx = tid + kCache * NT; idx < ncand; idx += NT) {
        const unsigned key = idx < nb ? stay_key(idx) : ext_key(idx);
        if (key) atomicAdd(&h[key >> 24], 1u);
        local_max = max(local_max, key);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1)
        local_max = max(local_max, __shfl_xor_sync(0xffffffffu, local_max, o));
      if ((tid & 31) == 0 && local_max) atomicMax(reinterpret_cast<unsigned*>(&S.scal[SC_MAXKEY]), local_max);
    }
    __syncthreads();  // B
    if (tid < 32) resolve_digit(S, 0, 24);
    __syncthreads();  // C

    auto cand_key = [&](int k, int idx) -> unsigned {
      (void)k;
      return idx < nb ? S.st_key[idx] : ext_key(idx);
    };

    for (int pass = 1; pass < kPasses; ++pass) {
      if (S.scal[SC_DONE]) break;  // block-uniform: written before the last barrier
      const int shift = 32 - kRadixBits * (pass + 1);
      const unsigned prefix = (unsigned)S.scal[SC_PREFIX];
      unsigned* h = S.hist + pass * kBins;
#pragma unroll
      for (int k = 0; k < kCache; ++k) {
        const unsigned key = kc[k];
        if (key && (key >> (shift + kRadixBits)) == prefix) atomicAdd(&h[(key >> shift) & (kBins - 1)], 1u);
      }
      for (int idx = tid + kCache * NT; idx < ncand; idx += NT) {
        const unsigned key = cand_key(0, idx);
        if (key && (key >> (shift + kRadixBits)) == prefix) atomicAdd(&h[(key >> shift) & (kBins - 1)], 1u);
      }
      __syncthreads();
      if (tid < 32) resolve_digit(S, pass, shift);
      __syncthreads();
    }

    // P5: compaction of the selected candidates into the next beam
    const int shift = S.scal[SC_SHIFT];
    const unsigned prefix = (unsigned)S.scal[SC_PREFIX];
    const int need = S.scal[SC_NEED];
    const bool take_all = S.scal[SC_TAKEALL] != 0;
    const unsigned maxkey = (unsigned)S.scal[SC_MAXKEY];
    const int nbn = maxkey ? S.scal[SC_NBEAM_NEXT] : 0;
    const float best = maxkey ? key_score(maxkey) : 0.f;

    unsigned long long mine = 0ull;
    {
#pragma unroll
      for (int k = 0; k < kCache; ++k) {
        const unsigned key = kc[k];
        if (key) {
          const unsigned hk = key >> shift;
          mine += (hk > prefix) ? 1ull : ((hk == prefix) ? (1ull << 32) : 0ull);
        }
      }
      for (int idx = tid + kCache * NT; idx < ncand; idx += NT) {
        const unsigned key = cand_key(0, idx);
        if (key) {
          const unsigned hk = key >> shift;
          mine += (hk > prefix) ? 1ull : ((hk == prefix) ? (1ull << 32) : 0ull);
        }
      }
    }
    unsigned long long total;
    const unsigned long long excl = block_exclusive_scan(mine, S.warp_sums, &total);
    {
      int gt_rank = (int)(excl & 0xffffffffull), eq_rank = (int)(excl >> 32);
      const int total_gt = (int)(total & 0xffffffffull);
      auto place = [&](int idx, unsigned key) {
        int slot = -1;
        if (key) {
          const unsigned hk = key >> shift;
          if (hk > prefix) {
            slot = gt_rank++;
          } else if (hk == prefix) {
            if (take_all || eq_rank < need) slot = total_gt + eq_rank;
            ++eq_rank;
          }
        }
        if (idx < nb) {
          S.old2new[idx] = slot;
          if (slot >= 0) {
            N.node[slot] = C.node[idx]; N.last[slot] = C.last[idx];
            N.parnode[slot] = C.parnode[idx];
            N.pb[slot] = S.st_pb[idx] - best; N.pnb[slot] = S.st_pnb[idx] - best;
            N.first[slot] = C.first[idx]; N.len[slot] = C.len[idx]; N.filt[slot] = C.filt[idx];
            S.from[slot] = idx; S.isext[slot] = 0;
          }
        } else if (slot >= 0) {
          const int e = idx - nb;
          const int q = e / Snb;
          int j = e - q * Snb;
          if (blank_j >= 0 && j >= blank_j) ++j;
          N.node[slot] = -1; N.last[slot] = S.sv[buf][j].token;
          N.parnode[slot] = C.node[q];
          N.pb[slot] = neg_inf(); N.pnb[slot] = key_score(key) - best;
          N.first[slot] = -1; N.len[slot] = C.len[q] + 1; N.filt[slot] = 0ull;
          S.from[slot] = q; S.isext[slot] = 1;
        }
      };
#pragma unroll
      for (int k = 0; k < kCache; ++k) {
        const int idx = tid + k * NT;
        if (idx < ncand) place(idx, kc[k]);
      }
      for (int idx = tid + kCache * NT; idx < ncand; idx += NT) place(idx, cand_key(0, idx));
    }
    __syncthreads();  // D

    // P6a: parent slots of the next beam; look up children that may already exist
    for (int s = tid; s < nbn; s += NT) {
      const int q = S.from[s];
      if (S.isext[s]) {
        N.par[s] = S.old2new[q];
        const int tok = N.last[s];
        if ((C.filt[q] >> (tok & 63)) & 1ull) {
          int id = C.first[q];
          for (int it = 0; id >= 0 && it <= V; ++it) {
            const int4 rec = *reinterpret_cast<const int4*>(&nodes[id]);  // parent, token, first, next
            if (rec.y == tok) {
              N.node[s] = id;
              N.first[s] = rec.z;
              N.filt[s] = nodes[id].child_filter;
              S.scal[SC_REVIVED] = 1;
              break;
            }
            id = rec.w;
          }
        }
      } else {
        const int op = C.par[q];
        N.par[s] = op >= 0 ? S.old2new[op] : -1;
      }
    }
    __syncthreads();  // E

    // P6b: create the trie nodes of extensions seen for the first time
    for (int s = tid; s < nbn; s += NT) {
      if (S.isext[s] && N.node[s] < 0) {
        const int q = S.from[s];
        const int tok = N.last[s];
        const int id = n_nodes + s;
        if (id < p.nodes_per_utt) {
          const int prev = atomicExch(&C.first[q], id);
          atomicOr(&C.filt[q], 1ull << (tok & 63));
          S.dirty[q] = 1;
          TrieNode n;
          n.parent = C.node[q]; n.token = tok; n.first_child = -1; n.next_sibling = prev;
          n.depth = N.len[s]; n.pad = 0; n.child_filter = 0ull;
          nodes[id] = n;
          N.node[s] = id;
          ++created;
        } else {
          N.node[s] = 0;
          S.scal[SC_STATUS] = 2;  // FLTOP_ST_ARENA_FULL
        }
      }
    }
    __syncthreads();  // F

    // P6c: publish changed child lists, repair parent slots of revived prefixes, clean up
    for (int i = tid; i < nb; i += NT) {
      if (S.dirty[i]) {
        S.dirty[i] = 0;
        nodes[C.node[i]].first_child = C.first[i];
        nodes[C.node[i]].child_filter = C.filt[i];
        const int s = S.old2new[i];
        if (s >= 0) {
          N.first[s] = C.first[i];
          N.filt[s] = C.filt[i];
        }
      }
      const int par = C.par[i];
      if (par >= 0) S.inbeam[par * W + (C.last[i] >> 5)] = 0u;
    }
    if (S.scal[SC_REVIVED]) {
      for (int s = tid; s < nbn; s += NT) {
        if (S.isext[s] && N.node[s] < n_nodes) {
          const int x = N.node[s];
          for (int s2 = 0; s2 < nbn; ++s2)
            if (N.parnode[s2] == x) N.par[s2] = s;
        }
      }
    }
    for (int j = tid; j < Scur; j += NT) S.lpv[S.sv[buf][j].token] = neg_inf();
    if (tid == 0) S.scal[SC_BLANK_J] = -1;
    if (!maxkey) status |= 8;  // FLTOP_ST_EMPTY_BEAM
    offset += (double)best;
    n_nodes += nbn;
    live_sum += nbn;
    nb = nbn;
    cur ^= 1;
    cnt0 = cnt1;
    cnt1 = cnt2;
    cp_async_wait_all();
    __syncthreads();  // G
  }
  frames_seen += len;
  status |= S.scal[SC_STATUS];
  if (p.stats) {
    if (created) atomicAdd(&S.scal[SC_CREATED], created);
    __syncthreads();
    if (tid == 0) {
      int32_t* o = p.stats + 4 * (int64_t)b;
      o[0] = len; o[1] = S.scal[SC_CREATED]; o[2] = live_sum; o[3] = n_nodes;
    }
  }

  Beam& F = S.beam[cur];

  // ---- keep the beam for the next chunk (streaming) -----------------------------------
  if (p.streaming) {
    int32_t* a = st + kStateHeaderWords;
    for (int i = tid; i < nb; i += NT) {
      a[i] = F.node[i]; a[K + i] = F.last[i]; a[2 * K + i] = F.par[i]; a[3 * K + i] = F.parnode[i];
      a[4 * K + i] = __float_as_int(F.pb[i]); a[5 * K + i] = __float_as_int(F.pnb[i]);
      a[6 * K + i] = F.first[i]; a[7 * K + i] = F.len[i];
      reinterpret_cast<unsigned long long*>(a + 8 * K)[i] = F.filt[i];
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
    const int L = p.L;
    for (int i = tid; i < nb; i += NT) S.tot[i] = lse2(F.pb[i], F.pnb[i]);
    __syncthreads();
    bool truncated = false;
    for (int i = tid; i < nb; i += NT) {
      const float ti = S.tot[i];
      int rank = 0;
      for (int j = 0; j < nb; ++j) {
        const float tj = S.tot[j];
        rank += (tj > ti || (tj == ti && j < i)) ? 1 : 0;
      }
      const int64_t o = (int64_t)b * K + rank;
      p.out_scores[o] = (float)(offset + (double)ti);
      const int n = F.len[i];
      p.out_lens[o] = n;
      if (n > L) truncated = true;
      int32_t* dst = p.out_tokens + o * L;
      int node = F.node[i];
      for (int d = n - 1; d >= 0 && node > 0; --d) {
        const int2 rec = *reinterpret_cast<const int2*>(&nodes[node]);  // parent, token
        if (d < L) dst[d] = rec.y;
        node = rec.x;
      }
    }
    for (int k = nb + tid; k < K; k += NT) {
      p.out_lens[(int64_t)b * K + k] = 0;
      p.out_scores[(int64_t)b * K + k] = neg_inf();
    }
    if (truncated) atomicOr(&S.scal[SC_STATUS], 4);  // FLTOP_ST_TRUNCATED
    __syncthreads();
    status |= S.scal[SC_STATUS];
    if (tid == 0) p.out_nhyp[b] = nb;
  }
  if (tid == 0 && p.out_status) p.out_status[b] = status;
}

}  // namespace

size_t decode_smem_bytes(int K, int V) { return smem_layout(K, V, nullptr, nullptr); }

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
