// Device helpers shared by the CUDA translation units of the decode kernels: constants of the
// score histogram, score <-> key maps, log-sum-exp, prefix fingerprints and the warp scan
// that turns the score histogram into the cut.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace fltop {
namespace {

constexpr int kMaxThreads = 1024;
constexpr int kSmallBlock = 256;   // up to here every warp scans the histogram itself
constexpr int kMidBlock = 512;     // blocks up to here are compiled with 128 registers a thread
constexpr int kCache = 4;          // extension keys cached in registers per ext lane
static_assert(kCache == 4, "the cached-score selects in P3 are written out for four scores");
constexpr int kFastBins = 256;     // score histogram of the fast select
constexpr float kBinsPerNat = 4.f;
constexpr int kBinsPerLane = kFastBins / 32;
static_assert(kBinsPerLane == 8, "a lane reads its eight bins with two 128-bit loads");
constexpr int kListCap = 64;       // candidates of the cut bin ranked pairwise
constexpr int kRadixBits = 8;      // exact fallback select
constexpr int kBins = 1 << kRadixBits;
constexpr int kPasses = 32 / kRadixBits;
constexpr unsigned long long kRootPrint = 0x9E3779B97F4A7C15ull;
constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

// log(exp(a) + exp(b)); symmetric in its arguments.  The hardware exp2 / log2
// approximations are used: their absolute error (about 2e-7 per call) is of the
// order of one float32 rounding of the scores themselves.
__device__ __forceinline__ float lse2(float a, float b) {
  const float hi = fmaxf(a, b), lo = fminf(a, b);
  if (lo == neg_inf()) return hi;
#ifdef FLTOP_EXACT_LSE
  return hi + log1pf(expf(lo - hi));
#else
  return hi + __logf(1.f + __expf(lo - hi));
#endif
}

// Which utterance the calling block decodes in a launch of more blocks than SMs.  Blocks start
// in the order of their index, so handing the utterances out by length shortens the launch:
// the first `first_wave` blocks (one per SM) take the longest utterances, longest first, and
// the blocks that move in beside them take the rest from the shortest upwards, so that the
// longest frame chains share their SM for the shortest time.  Every block ranks all lengths
// itself (length descending, index ascending: the same permutation in every block).
// `scratch`: B + 1 ints of shared memory, free again on return.  All threads call.
__device__ __forceinline__ int utterance_by_length(const int32_t* lengths, int B, int T,
                                                   int first_wave, int* scratch) {
  const int tid = threadIdx.x, NT = blockDim.x;
  for (int i = tid; i < B; i += NT) {
    const int l = lengths[i];
    scratch[i] = (l < 0 || l > T) ? 0 : l;  // a bad length decodes nothing
  }
  __syncthreads();
  const int blk = blockIdx.x;
  const int want = blk < first_wave ? blk : B - 1 - (blk - first_wave);
  for (int u = tid; u < B; u += NT) {
    const int lu = scratch[u];
    int rank = 0;
    for (int v = 0; v < B; ++v) {
      const int lv = scratch[v];
      rank += (lv > lu || (lv == lu && v < u)) ? 1 : 0;
    }
    if (rank == want) scratch[B] = u;
  }
  __syncthreads();
  const int b = scratch[B];
  __syncthreads();
  return b;
}
constexpr int kByLengthMaxB = 1024;  // largest batch that is handed out by length

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
// Histogram bin of a score: monotone, bin 0 holds the best, the last bin
// everything below -(kFastBins-1)/kBinsPerNat.
__device__ __forceinline__ int score_bin(float s) {
  const int b = __float2int_rz(-s * kBinsPerNat);
  return min(kFastBins - 1, max(0, b));
}

// Fingerprint of a prefix extended by one token.
__device__ __forceinline__ unsigned long long child_print(unsigned long long h, int token) {
  unsigned long long x = (h ^ (unsigned long long)(unsigned)(token + 1)) * 0x9E3779B97F4A7C15ull;
  x ^= x >> 32;
  x *= 0xD6E8FEB86659FD93ull;
  x ^= x >> 32;
  return x;
}

// log(exp(a) + exp(b) + exp(c)): one pass, the three exponentials independent of one another.
__device__ __forceinline__ float lse3(float a, float b, float c) {
  const float hi = fmaxf(fmaxf(a, b), c);
  if (hi == neg_inf()) return hi;
  return hi + __logf(__expf(a - hi) + __expf(b - hi) + __expf(c - hi));
}

// What the scan of the score histogram says about the cut.
struct Cut {
  int thr;        // bin that holds the K-th best score; kFastBins if everything is kept
  int left;       // how many members of that bin are kept
  int cut_count;  // how many are in it
  int cut_base;   // candidates in better bins
  int total;      // candidates altogether
  int first;      // first lane whose group of bins is not empty (0 if there is no candidate)
};

// One warp turns the score histogram into the cut (all lanes get the result).
__device__ __forceinline__ Cut scan_score_histogram(const unsigned* hist, int K) {
  const int lane = threadIdx.x & 31;
  // lane l owns bins [8 l, 8 l + 8): inclusive prefix counts inside the lane, then over lanes
  const uint4 lo4 = reinterpret_cast<const uint4*>(hist)[2 * lane];
  const uint4 hi4 = reinterpret_cast<const uint4*>(hist)[2 * lane + 1];
  int pre[kBinsPerLane];
  pre[0] = (int)lo4.x; pre[1] = pre[0] + (int)lo4.y; pre[2] = pre[1] + (int)lo4.z;
  pre[3] = pre[2] + (int)lo4.w; pre[4] = pre[3] + (int)hi4.x; pre[5] = pre[4] + (int)hi4.y;
  pre[6] = pre[5] + (int)hi4.z; pre[7] = pre[6] + (int)hi4.w;
  const int c = pre[7];
  int inc = c;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int up = __shfl_up_sync(kFull, inc, o);
    if (lane >= o) inc += up;
  }
  const int before = inc - c;
  Cut r;
  const unsigned any = __ballot_sync(kFull, c != 0);
  r.first = any ? __ffs(any) - 1 : 0;
  r.total = __shfl_sync(kFull, inc, 31);
  if (r.total <= K) {
    r.thr = kFastBins; r.left = 0; r.cut_count = 0; r.cut_base = r.total;
    return r;
  }
  // The inclusive prefix counts grow with the bin, so the cut bin is the number of bins
  // whose count stays below K, the candidates above it are the largest such count, and the
  // bin's own population follows from the smallest count that reaches K.
  int n_below = 0, best_below = 0, first_reach = 0x7fffffff;
#pragma unroll
  for (int i = 0; i < kBinsPerLane; ++i) {
    const int v = before + pre[i];
    const bool below = v < K;
    n_below += below ? 1 : 0;
    best_below = below ? max(best_below, v) : best_below;
    first_reach = below ? first_reach : min(first_reach, v);
  }
  r.thr = __reduce_add_sync(kFull, n_below);
  r.cut_base = __reduce_max_sync(kFull, best_below);
  r.cut_count = __reduce_min_sync(kFull, first_reach) - r.cut_base;
  r.left = K - r.cut_base;
  return r;
}

// One warp turns the score histogram into the cut (all lanes get the result).  Lane l owns bins
// [8l, 8l + 8).  The prefix counts over lanes come from ballots over the bits of the lanes'
// counts (clamped to K, which leaves the place where the running count reaches K unchanged):
// independent instructions instead of a chain of shuffles.  KBITS: bits of K.
template <int KBITS>
__device__ __forceinline__ Cut scan_score_histogram_ballots(const unsigned* hist, int K) {
  const int lane = threadIdx.x & 31;
  const unsigned le_mask = 0xffffffffu >> (31 - lane);  // lanes up to and including this one
  {
    // Fast path: the K-th best score lies in the first 32 bins (within 8 nats of the
    // reference), one bin per lane.  This is the usual case: the reference follows the best.
    const int v = (int)hist[lane];
    const int vc = min(v, K);
    int inc1 = 0;
#pragma unroll
    for (int bit = 0; bit < KBITS; ++bit)
      inc1 += __popc(__ballot_sync(kFull, (vc >> bit) & 1) & le_mask) << bit;
    const unsigned reach1 = __ballot_sync(kFull, inc1 >= K);
    if (reach1) {
      const int owner = __ffs(reach1) - 1;
      const unsigned any1 = __ballot_sync(kFull, v != 0);
      Cut r;
      r.first = (__ffs(any1) - 1) >> 3;
      r.total = K;  // at least
      r.thr = owner;
      r.cut_base = __shfl_sync(kFull, inc1 - vc, owner);
      r.cut_count = __shfl_sync(kFull, v, owner);
      r.left = K - r.cut_base;
      return r;
    }
  }
  const uint4 lo4 = reinterpret_cast<const uint4*>(hist)[2 * lane];
  const uint4 hi4 = reinterpret_cast<const uint4*>(hist)[2 * lane + 1];
  int pre[kBinsPerLane];  // inclusive prefix counts inside the lane
  pre[0] = (int)lo4.x; pre[1] = (int)(lo4.x + lo4.y);
  pre[2] = pre[1] + (int)lo4.z; pre[3] = pre[1] + (int)(lo4.z + lo4.w);
  const int h01 = (int)(hi4.x + hi4.y), h23 = (int)(hi4.z + hi4.w);
  pre[4] = pre[3] + (int)hi4.x; pre[5] = pre[3] + h01;
  pre[6] = pre[5] + (int)hi4.z; pre[7] = pre[3] + (h01 + h23);
  const int c = pre[7];
  const int cc = min(c, K);
  int inc = 0;  // inclusive prefix of the clamped counts over lanes
#pragma unroll
  for (int bit = 0; bit < KBITS; ++bit)
    inc += __popc(__ballot_sync(kFull, (cc >> bit) & 1) & le_mask) << bit;
  const unsigned any = __ballot_sync(kFull, c != 0);
  const unsigned reach = __ballot_sync(kFull, inc >= K);
  Cut r;
  r.first = any ? __ffs(any) - 1 : 0;
  if (!reach) {  // fewer than K candidates: every one is kept (no count was clamped)
    r.total = __shfl_sync(kFull, inc, 31);
    r.thr = kFastBins; r.left = 0; r.cut_count = 0; r.cut_base = r.total;
    return r;
  }
  // The lane in which the running count reaches K: before it no count was clamped, so its
  // own prefix counts are exact.
  const int owner = __ffs(reach) - 1;
  const int before = inc - cc;
  int n_below = 0, base = before, at_cut = 0x7fffffff;
#pragma unroll
  for (int i = 0; i < kBinsPerLane; ++i) {
    const int v = before + pre[i];
    const bool below = v < K;
    n_below += below ? 1 : 0;
    base = below ? max(base, v) : base;
    at_cut = below ? at_cut : min(at_cut, v);
  }
  // thr in the top bits, the bin's population and the count above it below
  const unsigned packed = ((unsigned)n_below << 28) | ((unsigned)(at_cut - base) << 12) | (unsigned)base;
  const unsigned got = __shfl_sync(kFull, packed, owner);
  r.total = K;  // at least
  r.thr = owner * kBinsPerLane + (int)(got >> 28);
  r.cut_count = (int)((got >> 12) & 0xffffu);
  r.cut_base = (int)(got & 0xfffu);
  r.left = K - r.cut_base;
  return r;
}

}  // namespace
}  // namespace fltop
