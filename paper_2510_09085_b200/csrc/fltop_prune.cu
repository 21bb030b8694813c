// Frame-level token pruning (Algorithm 1, the conditional break; Section 3):
// a token survives a frame iff  logp >= logp_max + log R  (float32 add and
// compare).  Output per frame: the survivor count and the survivors as
// {token, logp} pairs in ascending token order.
//
// This is the one stage that streams the emissions from HBM.  A row is read
// exactly once with 128-bit loads, kept in registers while the row maximum is
// reduced with warp shuffles, and compacted with ballot + popc, so the kernel
// moves 4*V bytes in and 8*S + 4 bytes out per frame.  Emissions stored as
// fp16 or bf16 are widened to float32 on load (exact), so the comparison is
// the same float32 comparison and the row costs 2*V bytes.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>

#include "fltop_internal.h"

namespace fltop {
namespace {

constexpr int kPruneThreads = 256;

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

__device__ __forceinline__ bool row_is_live(const PruneParams& p, int64_t row, int& b, int& t) {
  // (a 64-bit division is a long instruction sequence: rows are numbered in 32 bits whenever
  // the batch allows it, which is always in practice)
  if ((int64_t)p.B * p.T < 0x7fffffffll) {
    b = (int)((unsigned)row / (unsigned)p.T);
    t = (int)((unsigned)row - (unsigned)b * (unsigned)p.T);
  } else {
    b = (int)(row / p.T);
    t = (int)(row - (int64_t)b * p.T);
  }
  int len = p.lengths[b];
  return len <= p.T && t < len;  // a negative or oversized length reads nothing
}

// Four consecutive emissions, widened to float32: one 16-byte or 8-byte streaming load.
__device__ __forceinline__ float4 load_quad(const float* src) {
  return __ldcs(reinterpret_cast<const float4*>(src));
}
__device__ __forceinline__ float4 load_quad(const __half* src) {
  const uint2 raw = __ldcs(reinterpret_cast<const uint2*>(src));
  const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
  const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
  return make_float4(lo.x, lo.y, hi.x, hi.y);
}
__device__ __forceinline__ float4 load_quad(const __nv_bfloat16* src) {
  const uint2 raw = __ldcs(reinterpret_cast<const uint2*>(src));
  const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
  const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
  return make_float4(lo.x, lo.y, hi.x, hi.y);
}
__device__ __forceinline__ float load_one(const float* src) { return *src; }
__device__ __forceinline__ float load_one(const __half* src) { return __half2float(*src); }
__device__ __forceinline__ float load_one(const __nv_bfloat16* src) { return __bfloat162float(*src); }

// LPR lanes cooperate on one row (LPR a power of two <= 32); every lane holds
// CH float4: tokens 4*LPR*i + 4*sub + j for i < CH, j < 4.  E: the stored element type.
template <typename E, int LPR, int CH>
__global__ void __launch_bounds__(kPruneThreads) prune_vec_kernel(PruneParams p) {
  constexpr int ROWS_PER_WARP = 32 / LPR;
  const int lane = threadIdx.x & 31;
  const int sub = lane % LPR;
  const int grp = lane / LPR;
  const unsigned grp_mask = (0xffffffffu >> (32 - LPR)) << (grp * LPR);
  const unsigned lt_mask = ((1u << sub) - 1u);  // lanes of my group before me
  const int64_t n_rows = (int64_t)p.B * p.T;
  const int64_t warp_global = (int64_t)blockIdx.x * (kPruneThreads / 32) + (threadIdx.x >> 5);
  const int64_t warp_stride = (int64_t)gridDim.x * (kPruneThreads / 32);

  for (int64_t row0 = warp_global * ROWS_PER_WARP; row0 < n_rows;
       row0 += warp_stride * ROWS_PER_WARP) {
    const int64_t row = row0 + grp;
    int b = 0, t = 0;
    const bool live = row < n_rows && row_is_live(p, row, b, t);
    float4 x[CH];
    float m = neg_inf();
    const E* src = static_cast<const E*>(p.logp) + (int64_t)b * p.stride_b + (int64_t)t * p.stride_t;
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int tok0 = 4 * LPR * i + 4 * sub;
      if (live && tok0 < p.V) {
        x[i] = load_quad(src + tok0);
      } else {
        x[i] = make_float4(neg_inf(), neg_inf(), neg_inf(), neg_inf());
      }
      m = fmaxf(m, fmaxf(fmaxf(x[i].x, x[i].y), fmaxf(x[i].z, x[i].w)));
    }
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    const float thr = __fadd_rn(m, p.log_r);

    Survivor* dst = p.entries + row * p.V;
    int base = 0;
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int tok0 = 4 * LPR * i + 4 * sub;
      const bool in = live && tok0 < p.V;
      const float v[4] = {x[i].x, x[i].y, x[i].z, x[i].w};
      bool k[4];
      unsigned bal[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        k[j] = in && v[j] >= thr;
        bal[j] = __ballot_sync(0xffffffffu, k[j]) & grp_mask;
      }
      // survivors of my group held by earlier lanes in this chunk
      const unsigned shifted_lt = lt_mask << (grp * LPR);
      int pos = base;
#pragma unroll
      for (int j = 0; j < 4; ++j) pos += __popc(bal[j] & shifted_lt);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (k[j]) {
          dst[pos] = Survivor{tok0 + j, v[j]};
          ++pos;
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) base += __popc(bal[j]);
    }
    if (sub == 0 && row < n_rows) p.counts[row] = base;
  }
}

// The same rows with far fewer instructions, for rows of at most eight float4 per lane
// (V <= 1024): a lane counts the survivors among its four tokens of every chunk, the counts of
// all chunks travel together as one 64-bit word (a byte per chunk) through ONE shuffle scan
// over the row's lanes, and each lane then knows where its survivors go.  Four ballots and
// eight population counts per chunk become two shuffles per scan step for the whole row; at
// V = 1024 that is about 300 instead of 1170 instructions a row, which is what it takes for
// the loads, not the issue slots, to set the pace.
template <typename E, int LPR, int CH>
__global__ void __launch_bounds__(kPruneThreads) prune_packed_kernel(PruneParams p) {
  static_assert(CH <= 8, "a byte per chunk in one 64-bit word");
  constexpr int ROWS_PER_WARP = 32 / LPR;
  const int lane = threadIdx.x & 31;
  const int sub = lane % LPR;
  const int grp = lane / LPR;
  const int64_t n_rows = (int64_t)p.B * p.T;
  const int64_t warp_global = (int64_t)blockIdx.x * (kPruneThreads / 32) + (threadIdx.x >> 5);
  const int64_t warp_stride = (int64_t)gridDim.x * (kPruneThreads / 32);

  for (int64_t row0 = warp_global * ROWS_PER_WARP; row0 < n_rows;
       row0 += warp_stride * ROWS_PER_WARP) {
    const int64_t row = row0 + grp;
    int b = 0, t = 0;
    const bool live = row < n_rows && row_is_live(p, row, b, t);
    float4 x[CH];
    float m = neg_inf();
    const E* src = static_cast<const E*>(p.logp) + (int64_t)b * p.stride_b + (int64_t)t * p.stride_t;
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int tok0 = 4 * LPR * i + 4 * sub;
      if (live && tok0 < p.V) {
        x[i] = load_quad(src + tok0);
      } else {
        x[i] = make_float4(neg_inf(), neg_inf(), neg_inf(), neg_inf());
      }
      m = fmaxf(m, fmaxf(fmaxf(x[i].x, x[i].y), fmaxf(x[i].z, x[i].w)));
    }
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    const float thr = __fadd_rn(m, p.log_r);

    // which of this lane's tokens survive (bit 4i + j), and how many per chunk (byte i)
    unsigned keep = 0u;
    unsigned long long cnt = 0ull;
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const bool in = live && 4 * LPR * i + 4 * sub < p.V;
      const unsigned k4 = (in && x[i].x >= thr ? 1u : 0u) | (in && x[i].y >= thr ? 2u : 0u) |
                          (in && x[i].z >= thr ? 4u : 0u) | (in && x[i].w >= thr ? 8u : 0u);
      keep |= k4 << (4 * i);
      cnt |= (unsigned long long)__popc(k4) << (8 * i);
    }
    // inclusive scan over the lanes of the row, all chunks at once (a chunk's count over a
    // whole row is at most 128: a byte holds it)
    unsigned long long inc = cnt;
#pragma unroll
    for (int o = 1; o < LPR; o <<= 1) {
      const unsigned long long up = __shfl_up_sync(0xffffffffu, inc, o, LPR);
      if (sub >= o) inc += up;
    }
    const unsigned long long tot = __shfl_sync(0xffffffffu, inc, LPR - 1, LPR);
    const unsigned long long before = inc - cnt;

    Survivor* dst = p.entries + row * p.V;
    int base = 0;
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int tok0 = 4 * LPR * i + 4 * sub;
      int pos = base + (int)((before >> (8 * i)) & 0xffu);
      const unsigned k4 = (keep >> (4 * i)) & 0xfu;
      if (k4 & 1u) dst[pos++] = Survivor{tok0, x[i].x};
      if (k4 & 2u) dst[pos++] = Survivor{tok0 + 1, x[i].y};
      if (k4 & 4u) dst[pos++] = Survivor{tok0 + 2, x[i].z};
      if (k4 & 8u) dst[pos++] = Survivor{tok0 + 3, x[i].w};
      base += (int)((tot >> (8 * i)) & 0xffu);
    }
    if (sub == 0 && row < n_rows) p.counts[row] = base;
  }
}

// ---- rows staged through shared memory by asynchronous bulk copies -------------------------
// The register kernels above hold a row in registers from the moment its loads are issued, so
// the rows in flight per SM are bounded by the register file (24 warps x one 4 KB row) and the
// kernel ends up waiting on latency, not on bandwidth.  Here every warp owns a ring of three
// row buffers in shared memory; one lane issues a bulk copy (cp.async.bulk, global -> shared,
// completion on an mbarrier; not multicast) for the row three turns ahead, and the warp works
// on a row once its barrier has flipped.  No register is tied up while a row travels, 48 rows
// per SM are in flight, and the rest is the packed-count compaction of the kernel above.
// Needs rows of at most 4 KB that start on 16-byte boundaries.
// Measured on B200 (subword batch, 113 k live rows of 4 KB): 200 us against 154 us for the
// register kernel above, fp16 rows no faster than float32 ones - what bounds it is the warp's
// own chain per row at 16 resident warps, not the copies.  It is therefore not what a call
// gets by itself: fltop_set_test_hook(FLTOP_HOOK_PRUNE_STAGING) selects it, for measurements.
constexpr int kBulkStages = 3;
constexpr int kBulkSpin = 1 << 18;   // bounded wait on a copy; running out is reported

__device__ __forceinline__ unsigned smem_addr(const void* ptr) {
  return (unsigned)__cvta_generic_to_shared(ptr);
}
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("{ .reg .b64 st; mbarrier.arrive.shared::cta.b64 st, [%0]; }\n" ::"r"(smem_addr(bar))
               : "memory");
}
__device__ __forceinline__ void mbar_expect(unsigned long long* bar, unsigned bytes) {
  asm volatile("{ .reg .b64 st; mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }\n" ::"r"(
                   smem_addr(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, unsigned bytes,
                                          unsigned long long* bar) {
  asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(
          smem_addr(smem_dst)),
      "l"(gmem_src), "r"(bytes), "r"(smem_addr(bar))
      : "memory");
}
// waits until the barrier's phase with this parity is over; false if the wait ran out
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity) {
  const unsigned addr = smem_addr(bar);
  for (int it = 0; it < kBulkSpin; ++it) {
    unsigned done;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }\n"
        : "=r"(done)
        : "r"(addr), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}

__device__ __forceinline__ float4 widen_quad(const float* src) {
  return *reinterpret_cast<const float4*>(src);
}
__device__ __forceinline__ float4 widen_quad(const __half* src) {
  const uint2 raw = *reinterpret_cast<const uint2*>(src);
  const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
  const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
  return make_float4(lo.x, lo.y, hi.x, hi.y);
}
__device__ __forceinline__ float4 widen_quad(const __nv_bfloat16* src) {
  const uint2 raw = *reinterpret_cast<const uint2*>(src);
  const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
  const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
  return make_float4(lo.x, lo.y, hi.x, hi.y);
}

// CH: float4 per lane (tokens 128 i + 4 lane + j), V <= 128 CH.
template <typename E, int CH>
__global__ void __launch_bounds__(kPruneThreads) prune_bulk_kernel(PruneParams p) {
  static_assert(CH <= 8, "a byte per chunk in one 64-bit word");
  extern __shared__ __align__(128) unsigned char bulk_smem[];
  constexpr int W = kPruneThreads / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned row_bytes = (unsigned)p.V * (unsigned)sizeof(E);
  const unsigned pitch = (row_bytes + 127u) & ~127u;
  unsigned char* const ring = bulk_smem + (size_t)warp * kBulkStages * pitch;
  unsigned long long* const bars =
      reinterpret_cast<unsigned long long*>(bulk_smem + (size_t)W * kBulkStages * pitch) +
      warp * kBulkStages;
  if (lane == 0) {
    for (int st = 0; st < kBulkStages; ++st) mbar_init(bars + st, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncwarp();

  // Rows are dealt out to the warps in runs of eight consecutive frames (of one utterance,
  // mostly): a warp then needs a new utterance length only every few rows, and that load is
  // made by the cursor that runs three turns ahead, where nobody waits for it.
  constexpr int kRun = 8;
  const int64_t n_rows = (int64_t)p.B * p.T;
  const int64_t n_warps = (int64_t)gridDim.x * W;
  const int64_t me = (int64_t)blockIdx.x * W + warp;
  struct Cursor {
    int64_t turn, row;
    int b, t, len;
  };
  auto place = [&](Cursor& c) {  // the row of turn c.turn (its run's first row: a division)
    c.row = ((c.turn / kRun) * n_warps + me) * kRun + (c.turn % kRun);
    if (c.row < n_rows) {
      if (c.turn % kRun == 0 || c.t + 1 >= p.T) {
        c.b = (int)(c.row / p.T);
        c.t = (int)(c.row - (int64_t)c.b * p.T);
        c.len = p.lengths[c.b];
      } else {
        ++c.t;
      }
    }
  };
  auto is_live = [&](const Cursor& c) -> bool { return c.len <= p.T && c.t < c.len; };
  // Requests the cursor's row into stage `st`.  A frame past its utterance's length is never
  // read: its barrier is simply arrived at, so that every turn flips its stage's phase.
  auto request = [&](const Cursor& c, int st) {
    if (lane != 0) return;
    if (is_live(c)) {
      const E* src = static_cast<const E*>(p.logp) + (int64_t)c.b * p.stride_b + (int64_t)c.t * p.stride_t;
      mbar_expect(bars + st, row_bytes);
      bulk_load(ring + (size_t)st * pitch, src, row_bytes, bars + st);
    } else {
      mbar_arrive(bars + st);
    }
  };
  Cursor ahead = Cursor{0, 0, 0, 0, 0}, at = Cursor{0, 0, 0, 0, 0};
  place(at);
  for (int k = 0; k < kBulkStages; ++k) {
    ahead.turn = k;
    place(ahead);
    if (ahead.row < n_rows) request(ahead, k);
  }
  // (a warp's rows grow with its turns: once one lies past the end, so do all that follow)
  bool failed = false;
  for (; at.row < n_rows; ++at.turn, place(at)) {
    const int64_t turn = at.turn, row = at.row;
    const int st = (int)(turn % kBulkStages);
    const unsigned parity = (unsigned)((turn / kBulkStages) & 1);
    if (!mbar_wait(bars + st, parity)) {
      failed = true;  // (all lanes see the same barrier: warp-uniform)
      break;
    }
    const bool live = is_live(at);
    const E* const buf = reinterpret_cast<const E*>(ring + (size_t)st * pitch);
    // first walk: the row maximum (the row stays in shared memory; nothing of it is kept in
    // registers, so the later walks index it freely)
    float m = neg_inf();
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int tok0 = 128 * i + 4 * lane;
      if (live && tok0 < p.V) {
        const float4 x = widen_quad(buf + tok0);
        m = fmaxf(m, fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w)));
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    const float thr = __fadd_rn(m, p.log_r);
    // second walk: which of this lane's tokens survive (bit 4i + j), how many per chunk (byte i)
    unsigned keep = 0u;
    unsigned long long cnt = 0ull;
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int tok0 = 128 * i + 4 * lane;
      if (live && tok0 < p.V) {
        const float4 x = widen_quad(buf + tok0);
        const unsigned k4 = (x.x >= thr ? 1u : 0u) | (x.y >= thr ? 2u : 0u) |
                            (x.z >= thr ? 4u : 0u) | (x.w >= thr ? 8u : 0u);
        keep |= k4 << (4 * i);
        cnt |= (unsigned long long)__popc(k4) << (8 * i);
      }
    }
    // one scan over the lanes for all chunks at once (a chunk's count over the row <= 128)
    unsigned long long inc = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long up = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += up;
    }
    const unsigned long long tot = __shfl_sync(0xffffffffu, inc, 31);
    const unsigned long long before = inc - cnt;
    // where each chunk's survivors start: 16 bits a chunk, four chunks a word
    unsigned long long start_lo = 0ull, start_hi = 0ull;
    int base = 0;
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      if (i < 4) start_lo |= (unsigned long long)base << (16 * i);
      else start_hi |= (unsigned long long)base << (16 * (i - 4));
      base += (int)((tot >> (8 * i)) & 0xffu);
    }
    // third walk: this lane's survivors, one per turn, each straight to its place
    Survivor* dst = p.entries + row * p.V;
    for (unsigned left = keep; left; left &= left - 1) {
      const int bit = __ffs(left) - 1;
      const int i = bit >> 2, j = bit & 3;
      const int tok = 128 * i + 4 * lane + j;
      const unsigned long long starts = i < 4 ? start_lo : start_hi;
      const int pos = (int)((starts >> (16 * (i & 3))) & 0xffffu) + (int)((before >> (8 * i)) & 0xffu) +
                      __popc(keep & ((1u << bit) - 1u) & (0xfu << (4 * i)));
      float v;
      if constexpr (sizeof(E) == 4) v = reinterpret_cast<const float*>(buf)[tok];
      else v = load_one(buf + tok);
      dst[pos] = Survivor{tok, v};
    }
    // (the buffer is free only now: the third walk still read it)
    __syncwarp();
    ++ahead.turn;
    place(ahead);
    if (ahead.row < n_rows) request(ahead, st);
    if (lane == 0) p.counts[row] = base;
  }
  if (failed) {
    // A copy did not arrive within the bound: flag the call, give the copies that may still be
    // in flight a last bounded wait before the block's shared memory goes away, and count
    // nothing for the rows that are left.
    if (lane == 0 && p.error) atomicOr(p.error, 1);
    for (int64_t t2 = at.turn; t2 <= ahead.turn; ++t2)
      (void)mbar_wait(bars + (int)(t2 % kBulkStages), (unsigned)((t2 / kBulkStages) & 1));
    for (; at.row < n_rows; ++at.turn, place(at))
      if (lane == 0) p.counts[at.row] = 0;
  }
}

// Any V, any alignment: one warp per row, two passes over the row (the second
// pass is served by L1/L2).
template <typename E>
__global__ void __launch_bounds__(kPruneThreads) prune_scalar_kernel(PruneParams p) {
  const int lane = threadIdx.x & 31;
  const int64_t n_rows = (int64_t)p.B * p.T;
  const int64_t warp_global = (int64_t)blockIdx.x * (kPruneThreads / 32) + (threadIdx.x >> 5);
  const int64_t warp_stride = (int64_t)gridDim.x * (kPruneThreads / 32);
  for (int64_t row = warp_global; row < n_rows; row += warp_stride) {
    int b, t;
    const bool live = row_is_live(p, row, b, t);
    if (!live) {
      if (lane == 0) p.counts[row] = 0;
      continue;
    }
    const E* src = static_cast<const E*>(p.logp) + (int64_t)b * p.stride_b + (int64_t)t * p.stride_t;
    float m = neg_inf();
    for (int c = lane; c < p.V; c += 32) m = fmaxf(m, load_one(src + c));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    const float thr = __fadd_rn(m, p.log_r);
    Survivor* dst = p.entries + row * p.V;
    int base = 0;
    for (int c0 = 0; c0 < p.V; c0 += 32) {
      const int c = c0 + lane;
      const float v = c < p.V ? load_one(src + c) : neg_inf();
      const bool k = c < p.V && v >= thr;
      const unsigned bal = __ballot_sync(0xffffffffu, k);
      if (k) dst[base + __popc(bal & ((1u << lane) - 1u))] = Survivor{c, v};
      base += __popc(bal);
    }
    if (lane == 0) p.counts[row] = base;
  }
}

// Stage 1 of Algorithm 1 (PartialSortDesc(logits[t], N)): a frame keeps at most its top_n most
// probable survivors; at a tie for the last place the lower token id wins.  One warp per
// frame that has more than top_n survivors: an 8-bit radix select over order-preserving
// integer keys finds the top_n-th largest log-probability, then the list is compacted in
// place (it stays in ascending token order).
__global__ void __launch_bounds__(kPruneThreads) topn_cap_kernel(PruneParams p, int top_n) {
  __shared__ unsigned hist_all[kPruneThreads / 32][256];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned* const h = hist_all[warp];
  const unsigned lt_mask = (1u << lane) - 1u;
  const int64_t n_rows = (int64_t)p.B * p.T;
  const int64_t warp_global = (int64_t)blockIdx.x * (kPruneThreads / 32) + warp;
  const int64_t warp_stride = (int64_t)gridDim.x * (kPruneThreads / 32);
  auto order_key = [](float v) -> unsigned {
    const unsigned u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  };
  for (int64_t row = warp_global; row < n_rows; row += warp_stride) {
    const int count = p.counts[row];
    if (count <= top_n) continue;  // warp-uniform
    Survivor* const list = p.entries + row * p.V;
    if (count <= 32 && top_n <= 8) {
      // short list, small N: one entry per lane, the best one leaves top_n times (a tie goes
      // to the earlier entry, i.e. the lower token id)
      Survivor s = Survivor{0, 0.f};
      unsigned long long mine = 0ull;  // 0 = not in the running
      if (lane < count) {
        s = list[lane];
        mine = ((unsigned long long)order_key(s.logp) << 8) | (unsigned)(63 - lane);
      }
      bool keep = false;
      for (int n = 0; n < top_n; ++n) {
        unsigned long long best = mine;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
          best = other > best ? other : best;
        }
        if (mine == best) {
          keep = true;
          mine = 0ull;
        }
      }
      const unsigned km = __ballot_sync(0xffffffffu, keep);
      if (keep) list[__popc(km & lt_mask)] = s;
      if (lane == 0) p.counts[row] = __popc(km);
      continue;
    }
    unsigned prefix = 0u;
    int need = top_n;  // how many of the keys that share `prefix` are still to be taken
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      for (int i = lane; i < 256; i += 32) h[i] = 0u;
      __syncwarp();
      for (int i = lane; i < count; i += 32) {
        const unsigned key = order_key(list[i].logp);
        if (pass == 0 || (key >> (shift + 8)) == prefix) atomicAdd(&h[(key >> shift) & 255u], 1u);
      }
      __syncwarp();
      // lane l owns digits 255 - 8l .. 248 - 8l, walked from the largest
      unsigned c = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) c += h[255 - (lane * 8 + i)];
      unsigned inc = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned up = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += up;
      }
      const unsigned hit = __ballot_sync(0xffffffffu, (int)inc >= need);
      const int owner = __ffs(hit) - 1;  // exists: the group holds at least `need` keys
      int digit = 0, left = 0;
      if (lane == owner) {
        unsigned acc = inc - c;
        digit = 255 - lane * 8;
        for (int i = 0; i < 8; ++i, --digit) {
          const unsigned n = h[digit];
          if ((int)(acc + n) >= need) break;
          acc += n;
        }
        left = need - (int)acc;
      }
      digit = __shfl_sync(0xffffffffu, digit, owner);
      need = __shfl_sync(0xffffffffu, left, owner);
      prefix = (prefix << 8) | (unsigned)digit;
      __syncwarp();
    }
    // keys above `prefix` all stay; of the keys equal to it, the first `need` in token order
    int out_pos = 0, eq_seen = 0;
    for (int base = 0; base < count; base += 32) {
      const int i = base + lane;
      Survivor s = Survivor{0, 0.f};
      unsigned key = 0u;
      if (i < count) {
        s = list[i];
        key = order_key(s.logp);
      }
      const bool eq = i < count && key == prefix;
      const unsigned eqm = __ballot_sync(0xffffffffu, eq);
      const bool keep = i < count && (key > prefix || (eq && eq_seen + __popc(eqm & lt_mask) < need));
      const unsigned km = __ballot_sync(0xffffffffu, keep);  // every lane has loaded its entry
      if (keep) list[out_pos + __popc(km & lt_mask)] = s;
      out_pos += __popc(km);
      eq_seen += __popc(eqm);
    }
    if (lane == 0) p.counts[row] = out_pos;
  }
}

template <typename E, int LPR, int CH>
cudaError_t launch_vec(const PruneParams& p, cudaStream_t s, int sms) {
  const int64_t n_rows = (int64_t)p.B * p.T;
  const int rows_per_block = (kPruneThreads / 32) * (32 / LPR);
  int64_t blocks = (n_rows + rows_per_block - 1) / rows_per_block;
  const int64_t cap = (int64_t)sms * 8;  // 8 resident blocks of 256 threads per SM
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  if constexpr (CH <= 8)
    prune_packed_kernel<E, LPR, CH><<<(unsigned)blocks, kPruneThreads, 0, s>>>(p);
  else
    prune_vec_kernel<E, LPR, CH><<<(unsigned)blocks, kPruneThreads, 0, s>>>(p);
  return cudaGetLastError();
}

template <typename E>
cudaError_t launch_prune_typed(const PruneParams& p, cudaStream_t s) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  // four elements at a time: rows have to start on a multiple of four elements' bytes
  const bool aligned = (p.V % 4 == 0) && (p.stride_b % 4 == 0) && (p.stride_t % 4 == 0) &&
                       ((reinterpret_cast<uintptr_t>(p.logp) & (4 * sizeof(E) - 1)) == 0);
  // rows of 1 to 4 KB on 16-byte boundaries go through the shared-memory ring
  const size_t row_bytes = (size_t)p.V * sizeof(E);
  const bool bulk_ok = row_bytes % 16 == 0 && row_bytes >= 1024 && row_bytes <= 4096 && p.V <= 1024 &&
                       (p.stride_b * sizeof(E)) % 16 == 0 && (p.stride_t * sizeof(E)) % 16 == 0 &&
                       (reinterpret_cast<uintptr_t>(p.logp) & 15u) == 0;
  if (bulk_ok && p.staged) {
    const size_t pitch = (row_bytes + 127) & ~(size_t)127;
    const size_t smem = (size_t)(kPruneThreads / 32) * kBulkStages * (pitch + 8);
    const int rows_per_block = kPruneThreads / 32;
    const int64_t n_rows = (int64_t)p.B * p.T;
    int64_t blocks = (n_rows + rows_per_block - 1) / rows_per_block;
    const int per_sm = (int)std::max<size_t>(1, std::min<size_t>(8, (200 * 1024) / (smem + 1024)));
    if (blocks > (int64_t)sms * per_sm) blocks = (int64_t)sms * per_sm;
    auto go = [&](auto kernel) -> cudaError_t {
      cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      kernel<<<(unsigned)blocks, kPruneThreads, smem, s>>>(p);
      return cudaGetLastError();
    };
    const int ch = (p.V + 127) / 128;
    if (ch <= 2) return go(prune_bulk_kernel<E, 2>);
    if (ch <= 4) return go(prune_bulk_kernel<E, 4>);
    return go(prune_bulk_kernel<E, 8>);
  }
  if (aligned) {
    const int quads = p.V / 4;
    if (quads <= 1) return launch_vec<E, 1, 1>(p, s, sms);
    if (quads <= 2) return launch_vec<E, 2, 1>(p, s, sms);
    if (quads <= 4) return launch_vec<E, 4, 1>(p, s, sms);
    if (quads <= 8) return launch_vec<E, 8, 1>(p, s, sms);
    if (quads <= 16) return launch_vec<E, 16, 1>(p, s, sms);
    if (quads <= 32) return launch_vec<E, 32, 1>(p, s, sms);
    if (quads <= 64) return launch_vec<E, 32, 2>(p, s, sms);
    if (quads <= 128) return launch_vec<E, 32, 4>(p, s, sms);
    if (quads <= 256) return launch_vec<E, 32, 8>(p, s, sms);
    if (quads <= 512) return launch_vec<E, 32, 16>(p, s, sms);
  }
  const int64_t n_rows = (int64_t)p.B * p.T;
  int64_t blocks = (n_rows + (kPruneThreads / 32) - 1) / (kPruneThreads / 32);
  if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
  prune_scalar_kernel<E><<<(unsigned)blocks, kPruneThreads, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prune(const PruneParams& p, cudaStream_t s) {
  if ((int64_t)p.B * p.T == 0) return cudaSuccess;
  switch (p.dtype) {
    case kEmissionF16: return launch_prune_typed<__half>(p, s);
    case kEmissionBF16: return launch_prune_typed<__nv_bfloat16>(p, s);
    default: return launch_prune_typed<float>(p, s);
  }
}

cudaError_t launch_topn_cap(const PruneParams& p, int top_n, cudaStream_t s) {
  const int64_t n_rows = (int64_t)p.B * p.T;
  if (n_rows == 0 || top_n <= 0 || top_n >= p.V) return cudaSuccess;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int64_t blocks = (n_rows + (kPruneThreads / 32) - 1) / (kPruneThreads / 32);
  if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
  topn_cap_kernel<<<(unsigned)blocks, kPruneThreads, 0, s>>>(p, top_n);
  return cudaGetLastError();
}

}  // namespace fltop
