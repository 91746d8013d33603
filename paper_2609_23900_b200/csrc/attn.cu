// Attention half of the tree verifier (sm_100a): ancestry-masked decode attention on tcgen05 with
// TMA-staged key/value tiles, the write of the tree's entries through the slot map, and the
// re-linearisation of the accepted path at publication (paper Sec. "One slot map governs attention
// and publication"; Algorithm 1, "remap KV").
//
// tree_attn_kernel.  One CTA (256 threads) takes one (sequence, KV head, 128-row query tile, key-range
// partition).  The query rows of all heads that share the KV head sit in one tile (row = head-in-group
// * N + node), so each staged key/value tile serves the whole group.  Per tile of 64 keys:
//
//   TMA       K tile [64 keys x 128] and V tile, 128-byte swizzle, two stages, one mbarrier per stage
//   tcgen05   S = Q K^T           (M 128, N 64, K 128; fp32 in tensor memory columns 0..63)
//   threads   row = tensor-memory lane; a row is shared by two threads (warps w and w+4): both read the
//             whole row for the running maximum, each turns its 32 keys into probabilities (exp2 in
//             fp32, visibility applied by selection, never by arithmetic on the masked logit), rounds
//             them to bf16 and stores them as the next A operand
//   tcgen05   O_tile = P V        (M 128, N 2 x 64, K 64; V is the MN-major B operand as it lies in
//             memory; fp32 in tensor memory columns 64..191)
//   threads   each adds its 64 of the 128 output columns to fp32 registers, rescaled when the running
//             maximum moved.  The next tile's S product is issued together with this tile's O product.
//
// Only tiles that reach past the committed context need a mask; the mask of node i over the physical
// suffix is a bit row built with the tree descriptor.  Value rows of positions nobody may read (padding
// slots, beyond the suffix) are zeroed in shared memory before the product, so that bytes outside the
// visible set cannot reach any output (0 x NaN).  A partition writes normalised partial outputs and
// base-2 log-sum-exps to scratch; attn_merge_kernel combines them in partition order.
//
// Every wait is bounded; a wait that runs out marks the sequence LUMO_SEQ_TIMEOUT and the CTA leaves
// through the normal exit (barriers stay uniform, tensor memory is freed).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "internal.h"

namespace lumo {

namespace {

constexpr int kDh = 128;
constexpr int kRows = 128;            // query rows per CTA = tensor-memory lanes
constexpr int kKeys = 64;             // keys per tile
constexpr int kThreads = 256;
constexpr int kStages = 2;
constexpr int kTmemCols = 256;        // S: columns 0..63, O tile: 64..191 (power-of-two allocation)
constexpr int kColO = 64;
constexpr uint32_t kSpinLimit = 1u << 24;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// shared memory map; the dynamic segment starts at offset 0 of the CTA's window (no static shared
// variables in this file), which the 128-byte swizzle needs 1024-aligned; checked at run time
constexpr int kOffQ = 0;              // 2 halves of dh x [128 rows x 128 B]
constexpr int kOffP = 32768;          // [128 rows x 128 B] probabilities, bf16
constexpr int kOffKV = 49152;         // per stage: K 2 halves x [64 keys x 128 B], then V the same
constexpr int kStageBytes = 32768;
constexpr int kOffSmall = kOffKV + kStages * kStageBytes;   // 114688
struct Small {
  unsigned long long full[kStages];
  unsigned long long bar_qk, bar_pv;
  uint32_t tmem_base;
  uint32_t timed_out;
};
constexpr int kSmemBytes = kOffSmall + 64;
static_assert(sizeof(Small) <= 64, "small block");
static_assert(2 * (kSmemBytes + 1024) <= 228 * 1024, "two CTAs must share an SM");


__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Bounded wait: false if the phase did not complete within the spin limit.
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity) {
  const uint32_t addr = smem_u32(bar);
  for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
    uint32_t done;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(done) : "r"(addr), "r"(parity) : "memory");
    if (done) return true;
  }
  return false;
}

// One box of a 4-d tiled tensor map (dh, KV head, position, cache row) into shared memory; completion
// is counted in bytes on `bar`.  c0 is 0 or 64 elements: a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, unsigned long long* bar, int c0, int c1,
                                            int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];\n"
      ::"r"(dst), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// shared-memory matrix descriptor, 128-byte swizzle
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
  d |= (uint64_t)(lbo >> 4) << 16;
  d |= (uint64_t)(sbo >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// instruction descriptor: bf16 x bf16 -> fp32; *_mn = 1 when the operand is MN-major
__host__ __device__ constexpr uint32_t umma_idesc(int M, int N, int a_mn, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
// byte offset of 16-byte chunk `chunk` (0..7) of row `row` in a 128-byte-swizzled tile of 128-byte rows
__device__ __forceinline__ uint32_t sw128(int row, int chunk) {
  return (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((chunk ^ (row & 7)) << 4));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&t);
}

__device__ __forceinline__ int seq_check(int ctx, int crow, int Ns, int n_rows, int max_pos) {
  if (crow < 0 || crow >= n_rows) return LUMO_SEQ_BAD_ROW;
  if (ctx < 0 || ctx > max_pos - Ns) return LUMO_SEQ_BAD_CTX;
  return LUMO_SEQ_OK;
}

__global__ void __launch_bounds__(kThreads, 2)
tree_attn_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, const AttnArgs a) {
  extern __shared__ __align__(1024) unsigned char smem[];
  Small& sm = *reinterpret_cast<Small*>(smem + kOffSmall);
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int split = blockIdx.x, hkv = blockIdx.y / a.RT, rt = blockIdx.y % a.RT, b = blockIdx.z;
  const int row = 32 * (warp & 3) + lane;   // tensor-memory lane = query row of the tile
  const int half = warp >> 2;               // key half in the softmax, dh half in the accumulation
  const int GN = a.G * a.N;
  const int rg = rt * kRows + row;          // row within the (sequence, KV head) group
  const bool row_ok = rg < GN;
  const int hl = row_ok ? rg / a.N : 0, node = row_ok ? rg - hl * a.N : 0;

  const int ctx = a.ctx_len[b], crow = a.cache_row[b];
  int bad = seq_check(ctx, crow, a.Ns, a.n_rows, a.max_pos);
  if ((sbase & 1023u) != 0) bad = LUMO_SEQ_TIMEOUT;   // cannot happen with this file's layout; refuse rather than mis-swizzle
  const size_t out_row = (((size_t)b * a.N + node) * a.Hq + (size_t)hkv * a.G + hl);
  const size_t part_row = ((((size_t)b * a.Hkv + hkv) * a.RT + rt) * a.S + split) * kRows + row;
  if (bad != LUMO_SEQ_OK) {                 // uniform over the CTA: nothing was allocated or issued yet
    if (a.status && split == 0 && blockIdx.y == 0 && tid == 0) a.status[b] = bad;
    if (row_ok && split == 0) {
      float4* o = reinterpret_cast<float4*>(a.out + out_row * kDh + half * 64);
      for (int e = 0; e < 16; ++e) o[e] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (a.lse && half == 0) a.lse[out_row] = 0.f;
    }
    return;
  }

  // key tiles of this partition
  const int T = ctx + a.Ns;
  const int nt = (T + kKeys - 1) / kKeys;
  const int t0 = (int)(((long long)split * nt) / a.S), t1 = (int)(((long long)(split + 1) * nt) / a.S);
  const int n = t1 - t0;

  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&sm.tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(&sm.full[s], 1);
    mbar_init(&sm.bar_qk, 1);
    mbar_init(&sm.bar_pv, 1);
    sm.timed_out = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  // query tile: 128 rows x 16 chunks of 16 bytes, zero rows beyond the group
  for (int c = tid; c < kRows * 16; c += kThreads) {
    const int r = c >> 4, ch = c & 15;
    const int g = rt * kRows + r;
    uint4 val = make_uint4(0u, 0u, 0u, 0u);
    if (g < GN) {
      const int h = g / a.N, i = g - h * a.N;
      val = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(a.q) + ((((size_t)b * a.N + i) * a.Hq + (size_t)hkv * a.G + h) * kDh + ch * 8)));
    }
    *reinterpret_cast<uint4*>(smem + kOffQ + (ch >> 3) * 16384 + sw128(r, ch & 7)) = val;
  }
  fence_async_proxy();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  const uint32_t tmem_lane = tmem + ((uint32_t)(32 * (warp & 3)) << 16);

  // thread 0 is the producer (TMA) and the tensor-core issuer
  auto issue_tile = [&](int tile, int st) {
    mbar_expect_tx(&sm.full[st], kStageBytes);
    const uint32_t dst = sbase + kOffKV + st * kStageBytes;
    tma_load_4d(dst, &tm_k, &sm.full[st], 0, hkv, tile * kKeys, crow);
    tma_load_4d(dst + 8192, &tm_k, &sm.full[st], 64, hkv, tile * kKeys, crow);
    tma_load_4d(dst + 16384, &tm_v, &sm.full[st], 0, hkv, tile * kKeys, crow);
    tma_load_4d(dst + 24576, &tm_v, &sm.full[st], 64, hkv, tile * kKeys, crow);
  };
  auto issue_qk = [&](int st) {
    constexpr uint32_t id = umma_idesc(kRows, kKeys, 0, 0);
    const uint32_t kb = sbase + kOffKV + st * kStageBytes;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks)
      umma(tmem, umma_desc(sbase + kOffQ + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024),
           umma_desc(kb + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024), id, ks ? 1u : 0u);
    umma_commit(&sm.bar_qk);
  };
  auto issue_pv = [&](int st) {
    constexpr uint32_t id = umma_idesc(kRows, 64, 0, 1);
    const uint32_t vb = sbase + kOffKV + st * kStageBytes + 16384;
#pragma unroll
    for (int hh = 0; hh < 2; ++hh)
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)
        umma(tmem + kColO + hh * 64, umma_desc(sbase + kOffP + ks * 32, 16, 1024),
             umma_desc(vb + hh * 8192 + ks * 2048, 8192, 1024), id, ks ? 1u : 0u);
    umma_commit(&sm.bar_pv);
  };

  bool ok = true;
  int issued = 0;                           // tiles whose loads thread 0 has issued
  if (tid == 0) {
    for (; issued < n && issued < kStages; ++issued) issue_tile(t0 + issued, issued);
    if (n > 0) {
      ok = mbar_wait(&sm.full[0], 0);
      tc_fence_after();
      issue_qk(0);
    }
  }

  const uint32_t* visw = a.vis + ((size_t)b * a.N + node) * 8;
  const uint32_t* usedw = a.used + (size_t)b * 8;
  const float sl2 = a.scale_log2;
  float m = -INFINITY, l = 0.f;
  float o[64];
#pragma unroll
  for (int e = 0; e < 64; ++e) o[e] = 0.f;
  uint32_t ph_qk = 0, ph_pv = 0;

  for (int jj = 0; jj < n; ++jj) {
    const int st = jj & 1;
    const int kpos0 = (t0 + jj) * kKeys;
    const bool tail = kpos0 + kKeys > ctx;   // uniform: the tile reaches past the committed context
    // visibility of this row over the tile's 64 keys
    unsigned long long vm = row_ok ? ~0ull : 0ull;
    if (tail && row_ok) {
      vm = 0ull;
      for (int c = 0; c < kKeys; ++c) {
        const int p = kpos0 + c;
        bool v = p < ctx;
        if (!v) {
          const int s = p - ctx;
          if (s < a.Ns) v = (__ldg(visw + (s >> 5)) >> (s & 31)) & 1u;
        }
        vm |= (unsigned long long)v << c;
      }
    }
    if (ok) ok = mbar_wait(&sm.bar_qk, ph_qk);
    ph_qk ^= 1u;
    tc_fence_after();
    __syncwarp();                            // the tensor-memory loads below are warp-collective

    // pass 1: running maximum over the whole row
    float mx = -INFINITY;
#pragma unroll
    for (int c4 = 0; c4 < 4; ++c4) {
      uint32_t r[16];
      tmem_ld16(tmem_lane + c4 * 16, r);
      const uint32_t bits = (uint32_t)(vm >> (c4 * 16));
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const float s = __uint_as_float(r[e]);
        mx = fmaxf(mx, ((bits >> e) & 1u) ? s : -INFINITY);
      }
    }
    const float m_new = fmaxf(m, mx * sl2);
    const float m_use = m_new == -INFINITY ? 0.f : m_new;
    const float corr = ex2(m - m_use);       // m = -inf: 0
    m = m_new;
    l *= corr;
#pragma unroll
    for (int e = 0; e < 64; ++e) o[e] *= corr;
    // pass 2: this thread's 32 keys -> probabilities, bf16, A operand of the second product
    float lsum = 0.f;
#pragma unroll
    for (int c2 = 0; c2 < 2; ++c2) {
      uint32_t r[16];
      tmem_ld16(tmem_lane + half * 32 + c2 * 16, r);
      const uint32_t bits = (uint32_t)(vm >> (half * 32 + c2 * 16));
      uint32_t pk[8];
#pragma unroll
      for (int e = 0; e < 16; e += 2) {
        const float p0 = ((bits >> e) & 1u) ? ex2(fmaf(__uint_as_float(r[e]), sl2, -m_use)) : 0.f;
        const float p1 = ((bits >> (e + 1)) & 1u) ? ex2(fmaf(__uint_as_float(r[e + 1]), sl2, -m_use)) : 0.f;
        lsum += p0 + p1;
        pk[e >> 1] = pack_bf16(p0, p1);
      }
      const int chunk = half * 4 + c2 * 2;
      *reinterpret_cast<uint4*>(smem + kOffP + sw128(row, chunk)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
      *reinterpret_cast<uint4*>(smem + kOffP + sw128(row, chunk + 1)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
    }
    l += lsum;

    if (tail) {
      // value rows nobody may read: zero them in the staged tile (two 128-byte rows per key)
      if (ok) ok = mbar_wait(&sm.full[st], (uint32_t)(jj >> 1) & 1u);
      if (tid < 2 * kKeys) {
        const int c = tid >> 1, hh = tid & 1;
        const int p = kpos0 + c;
        bool dead = false;
        if (p >= ctx) {
          const int s = p - ctx;
          dead = s >= a.Ns || !((__ldg(usedw + (s >> 5)) >> (s & 31)) & 1u);
        }
        if (dead) {
          uint4* vrow = reinterpret_cast<uint4*>(smem + kOffKV + st * kStageBytes + 16384 + hh * 8192 + c * 128);
#pragma unroll
          for (int e = 0; e < 8; ++e) vrow[e] = make_uint4(0u, 0u, 0u, 0u);
        }
      }
    }
    fence_async_proxy();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      issue_pv(st);
      if (jj + 1 < n) {                      // next tile's logits run under this tile's accumulation
        if (ok) ok = mbar_wait(&sm.full[st ^ 1], (uint32_t)((jj + 1) >> 1) & 1u);
        tc_fence_after();
        issue_qk(st ^ 1);
      }
    }
    if (ok) ok = mbar_wait(&sm.bar_pv, ph_pv);
    ph_pv ^= 1u;
    tc_fence_after();
    if (tid == 0 && issued < n) {            // both products of this stage have completed: refill it
      issue_tile(t0 + issued, st);
      ++issued;
    }
    __syncwarp();
#pragma unroll
    for (int c4 = 0; c4 < 4; ++c4) {
      uint32_t r[16];
      tmem_ld16(tmem_lane + kColO + half * 64 + c4 * 16, r);
#pragma unroll
      for (int e = 0; e < 16; ++e) o[c4 * 16 + e] += __uint_as_float(r[e]);
    }
  }

  // after a wait that ran out, loads may still be in flight: give them a bounded chance to land
  if (tid == 0 && !ok)
    for (int t = 0; t < issued; ++t) (void)mbar_wait(&sm.full[t & 1], (uint32_t)(t >> 1) & 1u);
  if (!ok) sm.timed_out = 1u;
  tc_fence_before();
  __syncthreads();
  // the two halves of a row hold partial sums of the same scale (same running maximum)
  float* lbuf = reinterpret_cast<float*>(smem + kOffP);
  lbuf[half * kRows + row] = l;
  __syncthreads();
  const float lt = lbuf[row] + lbuf[kRows + row];
  const float inv = lt > 0.f ? 1.f / lt : 0.f;
  const float lse2 = lt > 0.f ? m + log2f(lt) : -INFINITY;
  if (row_ok) {
    float4* dst = a.S == 1 ? reinterpret_cast<float4*>(a.out + out_row * kDh + half * 64)
                           : reinterpret_cast<float4*>(a.part_o + part_row * kDh + half * 64);
#pragma unroll
    for (int e = 0; e < 16; ++e)
      dst[e] = make_float4(o[4 * e] * inv, o[4 * e + 1] * inv, o[4 * e + 2] * inv, o[4 * e + 3] * inv);
    if (half == 0) {
      if (a.S == 1) { if (a.lse) a.lse[out_row] = lse2 * kLn2; }
      else a.part_lse[part_row] = lse2;
    }
  }
  if (a.status && tid == 0) {
    if (sm.timed_out) a.status[b] = LUMO_SEQ_TIMEOUT;
    else if (split == 0 && blockIdx.y == 0) a.status[b] = LUMO_SEQ_OK;
  }
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

// Combination of the partitions' results: one warp per output row, partitions in index order (so the
// result for a given partition count is reproducible), weights exp2(lse_s - max lse).
__global__ void __launch_bounds__(256) attn_merge_kernel(const AttnArgs a) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int GN = a.G * a.N;
  const long long w = (long long)blockIdx.x * 8 + warp;
  if (w >= (long long)a.B * a.Hkv * GN) return;
  const int b = (int)(w / ((long long)a.Hkv * GN));
  const int rem = (int)(w - (long long)b * a.Hkv * GN);
  const int hkv = rem / GN, rg = rem - hkv * GN;
  const int rt = rg / kRows, r = rg - rt * kRows;
  const int hl = rg / a.N, node = rg - hl * a.N;
  const size_t out_row = (((size_t)b * a.N + node) * a.Hq + (size_t)hkv * a.G + hl);
  float4* dst = reinterpret_cast<float4*>(a.out + out_row * kDh) + lane;
  if (seq_check(a.ctx_len[b], a.cache_row[b], a.Ns, a.n_rows, a.max_pos) != LUMO_SEQ_OK) {
    *dst = make_float4(0.f, 0.f, 0.f, 0.f);
    if (a.lse && lane == 0) a.lse[out_row] = 0.f;
    return;
  }
  const size_t base = ((((size_t)b * a.Hkv + hkv) * a.RT + rt) * a.S) * kRows + r;
  float mx = -INFINITY;
  for (int s = 0; s < a.S; ++s) mx = fmaxf(mx, a.part_lse[base + (size_t)s * kRows]);
  float den = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s = 0; s < a.S; ++s) {
    const float ls = a.part_lse[base + (size_t)s * kRows];
    if (ls == -INFINITY) continue;
    const float wgt = ex2(ls - mx);
    const float4 v = reinterpret_cast<const float4*>(a.part_o + (base + (size_t)s * kRows) * kDh)[lane];
    den += wgt;
    acc.x = fmaf(wgt, v.x, acc.x); acc.y = fmaf(wgt, v.y, acc.y);
    acc.z = fmaf(wgt, v.z, acc.z); acc.w = fmaf(wgt, v.w, acc.w);
  }
  const float inv = den > 0.f ? 1.f / den : 0.f;
  *dst = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
  if (a.lse && lane == 0) a.lse[out_row] = den > 0.f ? (mx + log2f(den)) * kLn2 : -INFINITY;
}


// Scatter of the tree's entries: grid (node, sequence, layer); a CTA copies the Hkv x 128 keys and
// values of one node to position ctx + slot[node].
__global__ void __launch_bounds__(128) kv_write_kernel(const KvLayers L, const KvShape s) {
  const int i = blockIdx.x, b = blockIdx.y, l = blockIdx.z;
  const int ctx = s.ctx_len[b], crow = s.cache_row[b];
  const int bad = seq_check(ctx, crow, s.Ns, s.n_rows, s.max_pos);
  if (bad != LUMO_SEQ_OK) {
    if (L.status[l] && i == 0 && threadIdx.x == 0) L.status[l][b] = bad;
    return;
  }
  const int chunks = s.Hkv * kDh / 8;      // 16-byte chunks per entry
  const size_t src = ((size_t)b * s.N + i) * chunks;
  const size_t dst = ((size_t)crow * s.max_pos + ctx + s.slot[(size_t)b * s.N + i]) * chunks;
  const uint4* kn = reinterpret_cast<const uint4*>(L.kn[l]) + src;
  const uint4* vn = reinterpret_cast<const uint4*>(L.vn[l]) + src;
  uint4* kc = reinterpret_cast<uint4*>(L.k[l]) + dst;
  uint4* vc = reinterpret_cast<uint4*>(L.v[l]) + dst;
  for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
    kc[c] = __ldg(kn + c);
    vc[c] = __ldg(vn + c);
  }
}

// Publication: grid (KV head x {K, V}, sequence, layer).  A CTA stages the 256-byte pieces of all
// accepted entries that have to move (source != destination) in shared memory, then writes them: all
// reads come before any write, and pieces of different heads never overlap.
__global__ void __launch_bounds__(256) kv_publish_kernel(const KvLayers L, const KvShape s, const int32_t* __restrict__ accepted,
                                                         const int32_t* __restrict__ len, int lmax, int32_t* ctx_len_out) {
  extern __shared__ __align__(16) unsigned char stage[];     // [lmax][256 B]
  __shared__ int acc_s[kMaxNodes], par_s[kMaxNodes], src_s[kMaxNodes];
  __shared__ int st_s;
  const int hkv = blockIdx.x >> 1, which = blockIdx.x & 1, b = blockIdx.y, l = blockIdx.z;
  const int tid = threadIdx.x;
  const int ctx = s.ctx_len[b], crow = s.cache_row[b];
  const int n = len[b];
  const int nn = n < 0 ? 0 : (n > lmax ? lmax : n);
  for (int t = tid; t < nn; t += blockDim.x) {
    const int a = accepted[(size_t)b * lmax + t];
    acc_s[t] = a;
    const bool in = a >= 0 && a < s.N;
    par_s[t] = in ? s.parent[(size_t)b * s.N + a] : -2;
    src_s[t] = in ? s.slot[(size_t)b * s.N + a] : 0;
  }
  __syncthreads();
  if (tid == 0) {
    int st = seq_check(ctx, crow, s.Ns, s.n_rows, s.max_pos);
    if (st == LUMO_SEQ_OK) st = check_path_staged(acc_s, par_s, s.N, n, lmax);
    st_s = st;
    const bool lead = blockIdx.x == 0;
    if (lead && L.status[l]) L.status[l][b] = st;
    if (lead && l == 0 && ctx_len_out) ctx_len_out[b] = st == LUMO_SEQ_OK ? ctx + n : ctx;
  }
  __syncthreads();
  if (st_s != LUMO_SEQ_OK) return;
  unsigned char* cache = reinterpret_cast<unsigned char*>(which ? L.v[l] : L.k[l]);
  const size_t pos_bytes = (size_t)s.Hkv * kDh * 2;
  unsigned char* rowp = cache + ((size_t)crow * s.max_pos + ctx) * pos_bytes + (size_t)hkv * kDh * 2;
  // 16 chunks of 16 bytes per entry
  for (int c = tid; c < nn * 16; c += blockDim.x) {
    const int t = c >> 4, ch = c & 15;
    if (src_s[t] != t)
      reinterpret_cast<uint4*>(stage)[c] = *reinterpret_cast<const uint4*>(rowp + (size_t)src_s[t] * pos_bytes + ch * 16);
  }
  __syncthreads();
  for (int c = tid; c < nn * 16; c += blockDim.x) {
    const int t = c >> 4, ch = c & 15;
    if (src_s[t] != t)
      *reinterpret_cast<uint4*>(rowp + (size_t)t * pos_bytes + ch * 16) = reinterpret_cast<const uint4*>(stage)[c];
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map of one cache: dims (dh, KV head, position, row), box 64 x 1 x 64 x 1, 128-byte swizzle;
// positions beyond max_positions read as zeros.
cudaError_t encode_cache_map(void* cache, int Hkv, int max_pos, int n_rows, CUtensorMap* map, std::string* err) {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
    if (e != cudaSuccess) return e;
    if (q != cudaDriverEntryPointSuccess || !p) { *err = "the driver does not export cuTensorMapEncodeTiled"; return cudaErrorNotSupported; }
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  const cuuint64_t dims[4] = {(cuuint64_t)kDh, (cuuint64_t)Hkv, (cuuint64_t)max_pos, (cuuint64_t)n_rows};
  const cuuint64_t strides[3] = {(cuuint64_t)kDh * 2, (cuuint64_t)Hkv * kDh * 2, (cuuint64_t)max_pos * Hkv * kDh * 2};
  const cuuint32_t box[4] = {64, 1, (cuuint32_t)kKeys, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, cache, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { *err = "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r); return cudaErrorInvalidValue; }
  return cudaSuccess;
}

}  // namespace

int attn_row_tiles(int G, int N) { return (G * N + kRows - 1) / kRows; }

size_t attn_scratch_bytes(const AttnShape& s) {
  if (s.S <= 1) return 0;
  return (size_t)s.B * s.Hkv * attn_row_tiles(s.Hq / s.Hkv, s.N) * s.S * kRows * (kDh + 1) * sizeof(float);
}

cudaError_t attn_plan(const AttnShape& s, const AttnLayerPtrs& p, const uint32_t* vis, const uint32_t* used, float* scratch,
                      AttnPlan* plan, std::string* err) {
  static bool configured[kMaxDevices] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < kMaxDevices && !configured[dev]) {
    e = cudaFuncSetAttribute(tree_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  e = encode_cache_map(p.k_cache, s.Hkv, s.max_pos, s.n_rows, &plan->tk, err);
  if (e != cudaSuccess) return e;
  e = encode_cache_map(p.v_cache, s.Hkv, s.max_pos, s.n_rows, &plan->tv, err);
  if (e != cudaSuccess) return e;
  AttnArgs& a = plan->a;
  a.q = p.q;
  a.out = p.out; a.lse = p.lse;
  a.G = s.Hq / s.Hkv; a.RT = attn_row_tiles(a.G, s.N); a.S = s.S;
  a.part_o = scratch;
  a.part_lse = scratch ? scratch + (size_t)s.B * s.Hkv * a.RT * s.S * kRows * kDh : nullptr;
  a.ctx_len = s.ctx_len; a.cache_row = s.cache_row; a.vis = vis; a.used = used; a.status = p.status;
  a.B = s.B; a.N = s.N; a.Ns = s.Ns; a.Hq = s.Hq; a.Hkv = s.Hkv; a.n_rows = s.n_rows; a.max_pos = s.max_pos;
  a.scale_log2 = s.scale * kLog2e;
  plan->grid = dim3(s.S, s.Hkv * a.RT, s.B);
  return cudaSuccess;
}

cudaError_t launch_attn(const AttnPlan& plan, cudaStream_t st) {
  tree_attn_kernel<<<plan.grid, kThreads, kSmemBytes, st>>>(plan.tk, plan.tv, plan.a);
  return cudaGetLastError();
}

cudaError_t launch_attn_merge(const AttnPlan& plan, cudaStream_t st) {
  const long long rows = (long long)plan.a.B * plan.a.Hkv * plan.a.G * plan.a.N;
  attn_merge_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(plan.a);
  return cudaGetLastError();
}

cudaError_t launch_kv_write(const KvLayers& L, const KvShape& s, int n_layers, cudaStream_t st) {
  kv_write_kernel<<<dim3(s.N, s.B, n_layers), 128, 0, st>>>(L, s);
  return cudaGetLastError();
}

cudaError_t launch_kv_publish(const KvLayers& L, const KvShape& s, int n_layers, const int32_t* accepted, const int32_t* len,
                              int lmax, int32_t* ctx_len_out, cudaStream_t st) {
  static bool configured[kMaxDevices] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < kMaxDevices && !configured[dev]) {
    e = cudaFuncSetAttribute(kv_publish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxNodes * 256);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  kv_publish_kernel<<<dim3(2 * s.Hkv, s.B, n_layers), 256, (size_t)lmax * 256, st>>>(L, s, accepted, len, lmax, ctx_len_out);
  return cudaGetLastError();
}

}  // namespace lumo
