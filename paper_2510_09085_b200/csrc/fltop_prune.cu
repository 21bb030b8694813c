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

#include "fltop_internal.h"

namespace fltop {
namespace {

constexpr int kPruneThreads = 256;

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

__device__ __forceinline__ bool row_is_live(const PruneParams& p, int64_t row, int& b, int& t) {
  b = (int)(row / p.T);
  t = (int)(row - (int64_t)b * p.T);
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
