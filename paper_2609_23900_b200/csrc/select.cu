// Fused full-vocabulary draft selection (paper Sec. "Fuse draft selection without changing
// proposals"): one pass over a row of logits yields the spine token (argmax, lowest index among
// equal maxima) and three ordered sibling candidates (top-3 by value; among equal values the higher
// index first), written straight into caller-owned buffers.  The two tie conventions differ on
// purpose and both are kept; the candidates are not de-duplicated against the spine token, so
// candidate 0 repeats the spine token whenever the maximum is unique.
//
// One thread-block cluster per row, the vocabulary split over its CTAs; every thread keeps its own
// (max, three best) in registers; partial results merge through warp shuffles, shared memory and the
// peers' distributed shared memory.  Both orders are total, so the result does not depend on how the
// row was split (any cluster size gives the same bytes).
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <climits>

#include "internal.h"

namespace cg = cooperative_groups;

namespace lumo {

namespace {

constexpr int kSelThreads = 512;

// Both orders become plain unsigned comparisons of 64-bit keys: the high word is the value mapped
// monotonically to an unsigned integer (signed zeros made equal first), the low word the index for the
// candidate list (higher index first among equal values) or its complement for the spine token (lower
// index first).  Distinct indices make all keys of a row distinct; key 0 is below every real key.
using Key = unsigned long long;
__device__ __forceinline__ uint32_t ordered_bits(float v) {
  const uint32_t u = __float_as_uint(v + 0.0f);          // -0.0 + 0.0 = +0.0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float unordered_bits(uint32_t o) {
  return __uint_as_float((o & 0x80000000u) ? (o & 0x7FFFFFFFu) : ~o);
}
__device__ __forceinline__ Key kmax(Key a, Key b) { return a > b ? a : b; }
__device__ __forceinline__ Key kmin(Key a, Key b) { return a < b ? a : b; }

struct Best {
  Key s;             // spine
  Key t0, t1, t2;    // candidates, best first
  __device__ __forceinline__ void init() { s = t0 = t1 = t2 = 0; }
  __device__ __forceinline__ void push(float v, int i) {
    const Key hi = (Key)ordered_bits(v) << 32;
    s = kmax(s, hi | (0xFFFFFFFFu - (uint32_t)i));
    const Key c = hi | (uint32_t)i;
    const Key x = kmin(t0, c);
    t0 = kmax(t0, c);
    const Key y = kmin(t1, x);
    t1 = kmax(t1, x);
    t2 = kmax(t2, y);
  }
  // top three of two sorted triples
  __device__ __forceinline__ void merge(const Best& o) {
    s = kmax(s, o.s);
    const Key c0 = kmax(t0, o.t0), d0 = kmin(t0, o.t0), c1 = kmax(t1, o.t1), c2 = kmax(t2, o.t2);
    t0 = c0;
    t1 = kmax(d0, c1);
    t2 = kmax(kmin(d0, c1), c2);
  }
  // value of the weakest candidate: an entry below it changes nothing (entries are visited in
  // ascending index order, so an entry equal to the spine value never displaces the spine either)
  __device__ __forceinline__ float threshold() const {
    return t2 == 0 ? __int_as_float(0xff800000) : unordered_bits((uint32_t)(t2 >> 32));
  }
};

__device__ __forceinline__ void warp_merge(Best& b) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Best other;
    other.s = __shfl_xor_sync(0xffffffffu, b.s, o);
    other.t0 = __shfl_xor_sync(0xffffffffu, b.t0, o);
    other.t1 = __shfl_xor_sync(0xffffffffu, b.t1, o);
    other.t2 = __shfl_xor_sync(0xffffffffu, b.t2, o);
    b.merge(other);
  }
}

template <typename T> struct Vec;                       // 16 bytes of logits
template <> struct Vec<float> { static constexpr int n = 4; };
template <> struct Vec<__nv_bfloat16> { static constexpr int n = 8; };
__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const T* __restrict__ logits, int V, int32_t* __restrict__ spine, int32_t* __restrict__ cand) {
  __shared__ Best warp_best[kSelThreads / 32];
  __shared__ Best cta_best;
  __shared__ uint32_t cta_thr;                         // ordered bits of the best lower bound any warp has published
  cg::cluster_group cl = cg::this_cluster();
  const int rank = (int)cl.block_rank(), nblk = (int)cl.num_blocks();
  const int r = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const T* row = logits + (size_t)r * V;
  constexpr int n = Vec<T>::n;
  // the row's 16-byte units are dealt out to the CTAs in contiguous runs; a ragged head and tail
  // (row start not on a 16-byte boundary, V not a multiple of the unit) are read element by element
  const uintptr_t addr = reinterpret_cast<uintptr_t>(row);
  int head = (int)(((16 - (addr & 15)) & 15) / sizeof(T));
  if (head > V) head = V;
  const int units = (V - head) / n;
  const int tail0 = head + units * n;
  const int per = (units + nblk - 1) / nblk;
  const int u_lo = min(units, rank * per), u_hi = min(units, u_lo + per);
  if (tid == 0) cta_thr = ordered_bits(__int_as_float(0xff800000));
  __syncthreads();
  Best b;
  b.init();
  float thr = __int_as_float(0xff800000);              // -inf: everything passes until three entries are held
  constexpr int kU = 4;                                // independent 16-byte loads in flight per thread
  // The trip count is the same for every thread of the CTA (the warp-wide step below needs all lanes).
  const int iters = (u_hi - u_lo + kU * kSelThreads - 1) / (kU * kSelThreads);
  uint4 nxt[kU];                                       // the next iteration's units, requested one iteration ahead
  auto request = [&](int it) {
    const int u0 = u_lo + it * kU * kSelThreads + tid;
#pragma unroll
    for (int k = 0; k < kU; ++k) {
      const int u = u0 + k * kSelThreads;
      if (u < u_hi) nxt[k] = *reinterpret_cast<const uint4*>(row + head + (size_t)u * n);
    }
  };
  if (iters > 0) request(0);
  for (int it = 0; it < iters; ++it) {                 // bounded: units of this CTA
    const int u0 = u_lo + it * kU * kSelThreads + tid;
    uint4 raw[kU];
#pragma unroll
    for (int k = 0; k < kU; ++k) raw[k] = nxt[k];
    if (it + 1 < iters) request(it + 1);
    if (it == 0) {
      // Warm start: the third largest of the 32 lanes' maxima over their first units is reached by
      // three distinct entries, so it already bounds the row's third-best from below.
      uint32_t m = 0;
      {
        float mx = __int_as_float(0xff800000);
        bool have = false;
#pragma unroll
        for (int k = 0; k < kU; ++k)
          if (u0 + k * kSelThreads < u_hi) {
            const T* e = reinterpret_cast<const T*>(&raw[k]);
#pragma unroll
            for (int j = 0; j < n; ++j) mx = fmaxf(mx, to_f32(e[j]));
            have = true;
          }
        if (have) m = ordered_bits(mx);
      }
#pragma unroll
      for (int round = 0; round < 2; ++round) {
        const uint32_t top = __reduce_max_sync(0xffffffffu, m);
        const int owner = __ffs(__ballot_sync(0xffffffffu, m == top)) - 1;
        if (lane == owner) m = 0;
      }
      const uint32_t third = __reduce_max_sync(0xffffffffu, m);
      if (third != 0) thr = unordered_bits(third);
    } else {
      thr = fmaxf(thr, unordered_bits(cta_thr));       // what the other warps have found (may be stale: still a bound)
    }
#pragma unroll
    for (int k = 0; k < kU; ++k) {
      const int u = u0 + k * kSelThreads;
      if (u < u_hi) {
        if constexpr (sizeof(T) == 2) {
          // two entries per comparison; the threshold is a maximum of bf16 values, hence exact in bf16
          const __nv_bfloat162 thr2 = __float2bfloat162_rn(thr);
          const uint32_t w[4] = {raw[k].x, raw[k].y, raw[k].z, raw[k].w};
          bool any = false;
#pragma unroll
          for (int p = 0; p < 4; ++p) any |= __hge2_mask(*reinterpret_cast<const __nv_bfloat162*>(&w[p]), thr2) != 0;
          if (any) {
#pragma unroll
            for (int p = 0; p < 4; ++p) {
              const float lo = __uint_as_float(w[p] << 16), hi = __uint_as_float(w[p] & 0xFFFF0000u);
              if (lo >= thr) { b.push(lo, head + u * n + 2 * p); thr = fmaxf(thr, b.threshold()); }
              if (hi >= thr) { b.push(hi, head + u * n + 2 * p + 1); thr = fmaxf(thr, b.threshold()); }
            }
          }
        } else {
          const T* e = reinterpret_cast<const T*>(&raw[k]);
#pragma unroll
          for (int j = 0; j < n; ++j) {
            const float v = to_f32(e[j]);
            if (v >= thr) { b.push(v, head + u * n + j); thr = fmaxf(thr, b.threshold()); }
          }
        }
      }
    }
    // Any lane's third-best value bounds the row's third-best from below, so the largest of them
    // serves the whole warp: far fewer entries reach the slow path.
    const uint32_t wthr = __reduce_max_sync(0xffffffffu, ordered_bits(thr));
    thr = unordered_bits(wthr);
    if (lane == 0) atomicMax(&cta_thr, wthr);
  }
  if (rank == 0) {     // visited after the body, out of index order: no threshold shortcut here
    for (int i = tid; i < head; i += kSelThreads) b.push(to_f32(row[i]), i);
    for (int i = tail0 + tid; i < V; i += kSelThreads) b.push(to_f32(row[i]), i);
  }
  warp_merge(b);
  if (lane == 0) warp_best[warp] = b;
  __syncthreads();
  if (warp == 0) {
    if (lane < kSelThreads / 32) b = warp_best[lane]; else b.init();
    warp_merge(b);
    if (lane == 0) cta_best = b;
  }
  cl.sync();
  if (rank == 0 && warp == 0) {
    if (lane < nblk) b = *cl.map_shared_rank(&cta_best, lane); else b.init();
    warp_merge(b);
    if (lane == 0) {
      spine[r] = (int32_t)(0xFFFFFFFFu - (uint32_t)b.s);
      cand[3 * r + 0] = (int32_t)(uint32_t)b.t0; cand[3 * r + 1] = (int32_t)(uint32_t)b.t1; cand[3 * r + 2] = (int32_t)(uint32_t)b.t2;
    }
  }
  cl.sync();                                           // no CTA leaves while rank 0 may still read it
}

}  // namespace

cudaError_t launch_select(const void* logits, int dtype, int rows, int V, int split, int32_t* spine, int32_t* cand,
                          cudaStream_t st) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  static int cache_f[64] = {}, cache_h[64] = {};
  const int cap = dtype == LUMO_BF16 ? max_cluster_ctas(select_kernel<__nv_bfloat16>, kSelThreads, cache_h)
                                     : max_cluster_ctas(select_kernel<float>, kSelThreads, cache_f);
  int cluster = split;
  if (cluster == 0) {                                    // few rows: spread each over more SMs
    cluster = cap;
    while (cluster > 1 && (long long)rows * cluster > 2LL * sms) cluster >>= 1;
    const int unit = dtype == LUMO_BF16 ? 8 : 4;
    while (cluster > 1 && V < cluster * kSelThreads * unit) cluster >>= 1;
  }
  if (cluster > cap) return cudaErrorInvalidConfiguration;
  if (dtype == LUMO_BF16)
    return launch_cluster_kernel(select_kernel<__nv_bfloat16>, dim3(cluster, rows), dim3(kSelThreads), cluster, st,
                                 reinterpret_cast<const __nv_bfloat16*>(logits), V, spine, cand);
  return launch_cluster_kernel(select_kernel<float>, dim3(cluster, rows), dim3(kSelThreads), cluster, st,
                               reinterpret_cast<const float*>(logits), V, spine, cand);
}

}  // namespace lumo
