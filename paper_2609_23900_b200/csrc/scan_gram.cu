// Tree scan in Gram form on the 5th-generation tensor cores (tcgen05 + TMEM), sm_100a.
//
// Exact algebra of the recurrence (paper Eq. 2-3), no approximation.  With k^, q^ the scaled
// key/query of a node, G(t,s) the product of alpha over the nodes after s up to t on the path to
// t, and g_t = G from the pre-tree state S0:
//
//   delta_t = beta_t ( v_t - g_t S0 k^_t - sum_{s strict ancestor of t} G(t,s) (k^_s . k^_t) delta_s )
//   o_t     = g_t S0 q^_t + sum_{s ancestor of t or t itself} G(t,s) (k^_s . q^_t) delta_s
//
// (the ancestor-masked triangular system the paper cites as prior art for tree verification).
// Only two dense products touch d^2 data, and both run on tcgen05.mma with fp32 accumulators in
// tensor memory:
//   P    = S0 [K | Q]^T      [128 value rows x 2*64 nodes], S0 split exactly into bf16 hi + lo
//   Gram = [K ; Q] K^T       [2*64 x 64], exact products of bf16 inputs
// Everything after that is O(depth) fp32 FMAs per (row, node) in sequential fp32 arithmetic along
// each path: nodes are ordered by depth, a thread owns one value row (= TMEM lane) of one node
// at a time, the deltas live in shared memory [node][row], and the tree is walked level by level
// (all nodes of one depth are independent), the nodes of a level dealt out to the eight warps,
// each lane carrying four adjacent value rows so that the per-node coefficient loads are shared.
// Per node the CTA first builds a 208-byte record (coefficients, ancestor offsets, output
// offset); a warp loads the record of its next node before the barrier that publishes the
// previous level, so that only the ancestors' deltas are fetched after it.
//
// A second tail (kDirect, below) replaces the level-by-level walk by a closed form: M = W (I + A)^-1 per
// node along its own root path, then one pass over right-hand sides; the host picks per descriptor.
//
// One CTA (256 threads) handles one (layer, sequence, value head) at a time; two CTAs per SM
// overlap one item's loads with the other's arithmetic.  Limits of this
// kernel: d = 128, bf16 operands, N <= 64 nodes, tree depth <= 16, no state snapshots; everything
// else takes the rank-1 kernel.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "internal.h"

namespace lumo {

namespace {

constexpr int kD = 128;
constexpr int kNT = 64;               // node tile
constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kTmemCols = 256;        // P: 128 columns, Gram: 64 columns (power of two allocation)
constexpr int kDumpStride = 65;       // floats per dumped Gram row (odd: conflict-free scalar stores by row)
constexpr uint32_t kSpinLimit = 1u << 24;

// one record per node, built once per item, read by the warp that owns the node in the solve
struct NodeRec {
  float wk[16];     // -beta_t G(t,a_j) (k^_aj . k^_t), 0 beyond the node's depth
  float wq[16];     //          G(t,a_j) (k^_aj . q^_t), 0 beyond the node's depth
  float c0k;        // beta_t g_t |k scale|: factor of the S0 k product
  float beta;
  float c0q;        // g_t |q scale|: factor of the S0 q product
  float wself;      // k^_t . q^_t
  uint32_t out_off; // element offset of this node's output row for value row 0
  uint32_t pad[3];
  uint16_t aoff[16]; // element offset of ancestor j's deltas in the delta array; beyond the depth: the zero row
  uint32_t pad2[4];  // 208 bytes = 13 x 16: consecutive records start 13 bank groups apart, so the
                     // 128-bit stores of eight neighbouring threads never meet in a bank
};
static_assert(sizeof(NodeRec) == 208, "record layout");

// shared memory map (bytes from a 1024-aligned base)
constexpr int kOffAhi = 0;                          // S0 hi: 2 k-blocks x [128 rows x 128 B], SW128
constexpr int kOffAlo = 32768;                      // S0 lo
constexpr int kOffKQ = 65536;                       // rows 0..63 = K, 64..127 = Q, 2 k-blocks, SW128
constexpr int kOffSmall = 98304;
// once the MMAs have completed, the S0 tiles and later the K/Q tile are dead; their space is reused:
constexpr int kOffDump = 0;                         // Gram [128][65] fp32; later S0 k^ products, then deltas, [65][128] fp32
constexpr int kOffRec = 34816;                      // NodeRec[64]
static_assert(128 * kDumpStride * 4 <= kOffRec, "Gram dump overflows its area");
constexpr int kOffV = kOffRec + kNT * (int)sizeof(NodeRec);   // 49152: V [64][128] bf16
constexpr int kOffPq = kOffKQ;                      // S0 q^ products [64][128] fp32
constexpr int kZeroRow = kNT * kD;                  // element offset of the all-zero delta row
static_assert((kNT + 1) * kD * 4 <= kOffRec, "delta array overflows the dump area");
static_assert(kOffV + kNT * kD * 2 <= kOffKQ, "aliased region overflows the S0 tiles");

struct Small {
  float alpha[kNT], beta[kNT], ks[kNT], qs[kNT];
  int32_t meta[kNT];                 // physical row | depth << 16 | emit << 24
  uint8_t anc[kNT][16];              // positions of the ancestors, root first
  float qq[kNT];                     // |q|^2 of each node when normalising
  uint8_t lvl[20];                   // lvl[d] = number of nodes of depth <= d
  uint32_t bad[2];                   // tensor-core tail: nodes whose right-hand side is not finite (bit per node; rare)
  alignas(16) uint32_t out_off[kNT]; // tensor-core tail: element offset of each node's output row, ~0u when another group emits it
  unsigned long long mbar;
  uint32_t tmem_base;
  uint32_t timed_out;
};
constexpr int kSmemBytes = kOffSmall + (int)sizeof(Small) + 1024;   // + alignment slack

// fused commit + verify: the previous cycle's accepted path and its operands for this (sequence, head)
struct PrevStage {
  int32_t acc[kFusedMaxPath], par[kFusedMaxPath], phys[kFusedMaxPath];
  float ks[kFusedMaxPath];           // key normalisation factor of each accepted node
  float2 gates[kFusedMaxPath];       // alpha, beta
  __align__(16) __nv_bfloat16 k[kFusedMaxPath][kD];
  __align__(16) __nv_bfloat16 v[kFusedMaxPath][kD];
};
constexpr int kOffPrev = kOffSmall + (((int)sizeof(Small) + 15) / 16) * 16;
constexpr int kSmemBytesFused = kOffPrev + (int)sizeof(PrevStage) + 1024;

// Layout of one CTA.  Compact (trees of at most 32 nodes, not fused): the state crosses shared memory
// one 64-column half at a time (hi + lo of one k-block, 32 KB), the aliased areas shrink with the node
// count, and a CTA needs 68 KB of shared memory and 128 tensor-memory columns: three CTAs per SM
// instead of two (and 80 registers per thread instead of 128).
template <bool C>
struct GL {
  static constexpr int kNodes = C ? 32 : kNT;
  static constexpr int kAhi = 0, kAlo = C ? 16384 : 32768;
  static constexpr int kKQ = C ? 32768 : kOffKQ;
  static constexpr int kSmall = C ? 65536 : kOffSmall;
  static constexpr int kStride = C ? 33 : kDumpStride;         // floats per dumped Gram row
  static constexpr int kRec = C ? 128 * 33 * 4 : kOffRec;      // records behind the Gram dump / the deltas
  static constexpr int kV = kRec + kNodes * (int)sizeof(NodeRec);
  static constexpr int kZero = kNodes * kD;                    // element offset of the all-zero delta row
  static constexpr int kTmem = C ? 128 : kTmemCols;
  static constexpr int kGramCol = C ? 64 : 128;                // first tensor-memory column of the Gram block
  static constexpr int kBytes = kSmall + (int)sizeof(Small) + 1024;
};
static_assert((GL<true>::kNodes + 1) * kD * 4 <= GL<true>::kRec, "delta array overflows the dump area");
static_assert(GL<true>::kV + GL<true>::kNodes * kD * 2 <= GL<true>::kKQ, "aliased region overflows the state tiles");
static_assert(3 * (GL<true>::kBytes + 1024) <= 228 * 1024, "three compact CTAs must share an SM");

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(gmem) : "memory");
}
// pull of the 128-byte line at `gmem` into L2 (a request without a destination register)
__device__ __forceinline__ void prefetch_l2(const void* gmem) {
  asm volatile("prefetch.global.L2 [%0];\n" ::"l"(gmem) : "memory");
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(count) : "memory");
  asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
}
// Bounded wait: returns false if the phase did not complete within the spin limit.
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

// K-major, 128-byte swizzle: rows of 128 B, 8-row groups 1024 B apart; version 1 (sm_100).
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);          // start address
  d |= (uint64_t)1 << 16;                           // leading byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;                 // stride byte offset
  d |= (uint64_t)1 << 46;                           // descriptor version
  d |= (uint64_t)2 << 61;                           // SWIZZLE_128B
  return d;
}
// kind::f16, bf16 x bf16 -> fp32, both operands K-major
__host__ __device__ constexpr uint32_t umma_idesc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
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
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }
// 32 consecutive columns of this thread's TMEM lane -> shared memory dst[col * stride]
__device__ __forceinline__ void tmem_cols32_to_smem(uint32_t taddr, float* dst, int stride) {
  uint32_t r0[16], r1[16];
  tmem_ld16_issue(taddr, r0);
  tmem_ld16_issue(taddr + 16, r1);
  tmem_ld_wait();
#pragma unroll
  for (int e = 0; e < 16; ++e) dst[e * stride] = __uint_as_float(r0[e]);
#pragma unroll
  for (int e = 0; e < 16; ++e) dst[(16 + e) * stride] = __uint_as_float(r1[e]);
}

__device__ __forceinline__ uint32_t sw128_offset(int row, int chunk16) {   // within one [rows x 128 B] k-block
  return (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((chunk16 ^ (row & 7)) << 4));
}

__device__ __forceinline__ void store_out(void* out, size_t idx, int dtype, float v) {
  if (dtype == LUMO_BF16) reinterpret_cast<__nv_bfloat16*>(out)[idx] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(out)[idx] = v;
}

// fp32 x -> bf16 hi + lo of four values, written to the two swizzled operand tiles
template <int kHi = kOffAhi, int kLo = kOffAlo>
__device__ __forceinline__ void split_store(unsigned char* smem, uint32_t off, float4 x) {
  __nv_bfloat162 h01 = __floats2bfloat162_rn(x.x, x.y), h23 = __floats2bfloat162_rn(x.z, x.w);
  const float2 f01 = __bfloat1622float2(h01), f23 = __bfloat1622float2(h23);
  __nv_bfloat162 l01 = __floats2bfloat162_rn(x.x - f01.x, x.y - f01.y);
  __nv_bfloat162 l23 = __floats2bfloat162_rn(x.z - f23.x, x.w - f23.y);
  *reinterpret_cast<uint2*>(smem + kHi + off) = make_uint2(*reinterpret_cast<uint32_t*>(&h01), *reinterpret_cast<uint32_t*>(&h23));
  *reinterpret_cast<uint2*>(smem + kLo + off) = make_uint2(*reinterpret_cast<uint32_t*>(&l01), *reinterpret_cast<uint32_t*>(&l23));
}

// what a warp needs for one node besides its ancestors' deltas
struct NodeOps {
  float4 m;        // c0k, beta, c0q, wself
  uint32_t out_off;
  uint2 vb;        // four bf16 values of v
  float4 pk, pq;   // S0 k^, S0 q^ for the lane's four rows
  float4 ck, cq;   // first four coefficients
  uint2 ao;        // first four ancestor offsets (16 bits each)
};

// Closed-form tail of one item, entered when the Gram block has been dumped to shared memory
// (dump[R][c]: R < NT the products K_R . K_c, NT <= R < 2 NT the products Q_(R-NT) . K_c), the V rows
// are on their way (cp.async) and S0 [K | Q]^T sits in tensor-memory columns [0, 2 NT).
//
// With a_0 .. a_(D-1) the path of node t (root first, t itself last), A[t][j] = beta_t G(t, a_j)
// (k^_aj . k^_t) for the strict ancestors and W[t][j] = G(t, a_j) (k^_aj . q^_t) for all of them, the
// deltas solve (I + A) delta = rhs with rhs_s = beta_s (v_s - g_s S0 k^_s), and
//   o_t = g_t S0 q^_t + sum_j M[t][j] rhs_(a_j),   M = W (I + A)^-1.
// A and (I + A)^-1 couple only nodes of one root path, so row t of M comes from a back substitution
// over that path alone: m[j] = W[t][j] - sum_(i > j) m[i] A[a_i][j].  Nothing here waits for another
// node: four barrier-separated phases, whatever the depth of the tree.
template <int NT, class LY>
__device__ __forceinline__ void direct_tail(const Shape& s, const LayerPtrs& L, Small& sm, unsigned char* smem, const float* dump,
                                            const __nv_bfloat16* Vs, uint32_t tmem_lane, int N, int b, int hv, int tid) {
  const int warp = tid >> 5, lane = tid & 31, grp = tid >> 7, vrow = tid & 127;
  float* Am = reinterpret_cast<float*>(smem + LY::kRec);        // [node][16], in the place of the records
  float* Wm = Am + NT * 16;
  float* Mm = Wm + NT * 16;
  static_assert(LY::kRec + NT * 16 * 4 * 3 <= LY::kV, "coefficient tables overflow the record area");
  float* Pq = reinterpret_cast<float*>(smem);                   // S0 q products [node][row], in the place of the dump
  float* Rh = reinterpret_cast<float*>(smem + LY::kKQ);         // right-hand sides [node][row], in the place of K and Q
  // ---- A and W along each node's ancestry: sixteen lanes per node (lane j = path entry j); G(t, a_j)
  //      is a suffix product of the alphas over the lanes ----------------------------------------------
  {
    const int j = tid & 15, ln = tid >> 4;
#pragma unroll
    for (int m = 0; m < NT / 16; ++m) {
      if (16 * m >= N) break;                                       // uniform
      const int pi = ln + 16 * m;
      const int D = pi < N ? ((sm.meta[pi] >> 16) & 0xFF) : 0;      // depth, 1..16 (the same in all 16 lanes)
      const bool in = j < D;
      const int a = sm.anc[pi][j];                                  // 0 beyond the depth
      float incl = in ? sm.alpha[a] : 1.f;
#pragma unroll
      for (int off = 1; off < 16; off <<= 1) {
        const float v = __shfl_down_sync(0xffffffffu, incl, off, 16);
        if (j + off < 16) incl *= v;
      }
      float excl = __shfl_down_sync(0xffffffffu, incl, 1, 16);      // product over the lanes above j
      if (j == 15) excl = 1.f;
      const float g_t = __shfl_sync(0xffffffffu, incl, 0, 16);      // product over the whole path
      float ksa = 1.f;
      if (s.l2norm && in) ksa = rsqrtf(dump[a * LY::kStride + a] + s.l2_eps);
      const float ks_t = __shfl_sync(0xffffffffu, ksa, D > 0 ? D - 1 : 0, 16);
      const float qs_t = s.l2norm ? s.scale * rsqrtf(sm.qq[pi] + s.l2_eps) : s.scale;
      const float b_t = sm.beta[pi];
      float kk = 0.f, qk = 0.f;
      if (in) { kk = dump[pi * LY::kStride + a]; qk = dump[(NT + pi) * LY::kStride + a]; }
      Am[pi * 16 + j] = j < D - 1 ? b_t * excl * ks_t * ksa * kk : 0.f;   // no entry for the node itself
      Wm[pi * 16 + j] = in ? qs_t * excl * ksa * qk : 0.f;
      if (j == 0) { sm.qs[pi] = g_t * qs_t; sm.ks[pi] = b_t * g_t * ks_t; }   // factors of S0 q and of S0 k
    }
  }
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");            // this thread's pieces of V
  __syncthreads();                                                  // A, W, V in place; the dump is dead
  // ---- M by back substitution, four lanes per node holding its sixteen entries ------------------------
  if (tid < 4 * NT) {                                               // whole warps
    const int pi = tid >> 2, q4 = tid & 3;
    const int D = pi < N ? ((sm.meta[pi] >> 16) & 0xFF) : 0;
    float4 w = *reinterpret_cast<const float4*>(Wm + pi * 16 + 4 * q4);
    const int Dw = __reduce_max_sync(0xffffffffu, D);
    for (int jh = Dw - 1; jh >= 1; --jh) {                          // bounded: <= 15 steps
      const int e = jh & 3;
      const float cand = e == 0 ? w.x : e == 1 ? w.y : e == 2 ? w.z : w.w;
      const float mval = __shfl_sync(0xffffffffu, cand, (lane & ~3) | (jh >> 2));
      if (jh < D) {
        const float4 ar = *reinterpret_cast<const float4*>(Am + sm.anc[pi][jh] * 16 + 4 * q4);
        w.x = fmaf(-mval, ar.x, w.x); w.y = fmaf(-mval, ar.y, w.y);
        w.z = fmaf(-mval, ar.z, w.z); w.w = fmaf(-mval, ar.w, w.w);
      }
    }
    *reinterpret_cast<float4*>(Mm + pi * 16 + 4 * q4) = w;
  }
  // ---- the S0 products leave tensor memory (lane = value row): the first half of the CTA turns the key
  //      products into right-hand sides, the second half moves the query products ----------------------
  if (grp == 0) {
    for (int cb = 0; cb < (N + 31) / 32; ++cb) {                    // bounded: <= 2
      uint32_t r0[16], r1[16];
      tmem_ld16_issue(tmem_lane + cb * 32, r0);
      tmem_ld16_issue(tmem_lane + cb * 32 + 16, r1);
      tmem_ld_wait();
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        const int sn = cb * 32 + e;
        const float pk = __uint_as_float(e < 16 ? r0[e & 15] : r1[e & 15]);
        const float v = __bfloat162float(Vs[sn * kD + vrow]);       // rows of padding nodes hold stale bytes: never read back
        Rh[sn * kD + vrow] = fmaf(sm.beta[sn], v, -sm.ks[sn] * pk);
      }
    }
  } else {
    for (int cb = 0; cb < (N + 31) / 32; ++cb)                      // bounded: <= 2
      tmem_cols32_to_smem(tmem_lane + NT + cb * 32, Pq + (cb * 32) * kD + vrow, kD);
  }
  __syncthreads();
  // ---- outputs: one warp per node, lane l carries value rows 4l .. 4l+3; a node that another group
  //      emits is skipped altogether ----------------------------------------------------------------------
  for (int pi = warp; pi < N; pi += kWarps) {                       // bounded: <= 8 rounds
    const int meta = sm.meta[pi];
    if (!((meta >> 24) & 1)) continue;
    const int D = (meta >> 16) & 0xFF;
    const float cq = sm.qs[pi];
    const float4 pq = *reinterpret_cast<const float4*>(Pq + pi * kD + 4 * lane);
    float2 o01 = make_float2(cq * pq.x, cq * pq.y), o23 = make_float2(cq * pq.z, cq * pq.w);
    const int nblk = (D + 3) >> 2;
    for (int blk = 0; blk < nblk; ++blk) {                          // bounded: <= 4 blocks of four path entries
      const float4 mc = *reinterpret_cast<const float4*>(Mm + pi * 16 + 4 * blk);
      const uint32_t a4 = *reinterpret_cast<const uint32_t*>(&sm.anc[pi][4 * blk]);
      // entries beyond the depth (last block only) have m = 0 and read the node's own row: nothing of
      // another branch can reach this output, not even as 0 x NaN
      const int rem = D - 4 * blk;
      const float4 d0 = *reinterpret_cast<const float4*>(Rh + (a4 & 0xFF) * kD + 4 * lane);
      const float4 d1 = *reinterpret_cast<const float4*>(Rh + (rem > 1 ? (a4 >> 8) & 0xFF : pi) * kD + 4 * lane);
      const float4 d2 = *reinterpret_cast<const float4*>(Rh + (rem > 2 ? (a4 >> 16) & 0xFF : pi) * kD + 4 * lane);
      const float4 d3 = *reinterpret_cast<const float4*>(Rh + (rem > 3 ? a4 >> 24 : pi) * kD + 4 * lane);
      auto step = [&](float m, const float4& dd) {
        const float2 mm = make_float2(m, m);
        o01 = __ffma2_rn(mm, make_float2(dd.x, dd.y), o01);
        o23 = __ffma2_rn(mm, make_float2(dd.z, dd.w), o23);
      };
      step(mc.x, d0); step(mc.y, d1); step(mc.z, d2); step(mc.w, d3);
    }
    const size_t oi = (((size_t)b * s.Ns + (meta & 0xFFFF)) * s.Hv + hv) * kD + 4 * lane;
    if (s.out_dtype == LUMO_BF16) {
      __nv_bfloat162 b01 = __floats2bfloat162_rn(o01.x, o01.y), b23 = __floats2bfloat162_rn(o23.x, o23.y);
      *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(L.out) + oi) =
          make_uint2(*reinterpret_cast<uint32_t*>(&b01), *reinterpret_cast<uint32_t*>(&b23));
    } else {
      *reinterpret_cast<float4*>(reinterpret_cast<float*>(L.out) + oi) = make_float4(o01.x, o01.y, o23.x, o23.y);
    }
  }
}

// Closed-form tail with the output sum on the tensor core.  Same scalar part as direct_tail (A, W, then
// M = W (I + A)^-1 per node along its own root path); the sum o_t = g_t |q scale| S0 q_t + sum_s M[t][s] rhs_s
// is then ONE product over all nodes of the group, O[row][t] = sum_s RHS[row][s] M[t][s] (M is zero off the
// path), with both operands split into bf16 hi + lo (three products: hi.hi + hi.lo + lo.hi, relative error
// 2^-16).  RHS [128 rows x NT nodes] and M [NT x NT] are K-major tiles with the 128-byte swizzle (a row of 64
// nodes is one swizzle row; with NT = 32 the hi and lo halves share a row).  The result lands in the tensor-
// memory columns of the Gram block and leaves lane = value row together with the query products.
// A dense product would let a non-finite right-hand side of ANY node reach every output of the group (0 x NaN),
// where the recurrence confines it to the node's subtree.  So a right-hand side that is not finite (or overflows
// bf16) enters the product as zero and marks its node; when any node is marked (rare), the outputs of exactly the
// nodes with a marked node on their path are written as NaN.  Non-finite keys, queries and gates need no such
// care: they reach M only in the rows of the node's descendants, and the query products only the node itself.
// Returns false when the bounded wait for the product ran out.
template <int NT, class LY, bool kCompact>
__device__ __forceinline__ bool direct_tail_tc(const Shape& s, const LayerPtrs& L, Small& sm, unsigned char* smem, uint32_t sbase,
                                               const float* dump, const __nv_bfloat16* Vs, uint32_t tmem, uint32_t tmem_lane,
                                               int N, int b, int hv, int tid, uint32_t& phase) {
  const int lane = tid & 31, grp = tid >> 7, vrow = tid & 127;
  float* Am = reinterpret_cast<float*>(smem + LY::kRec);        // [node][16], in the place of the records
  float* Wm = Am + NT * 16;
  static_assert(LY::kRec + NT * 16 * 4 * 2 <= LY::kV, "coefficient tables overflow the record area");
  constexpr int kRt = kCompact ? LY::kKQ : 0;                   // RHS tiles: over the dead Gram dump, or (compact) over K and Q
  constexpr int kMt = kCompact ? LY::kKQ + 16384 : LY::kKQ;     // M tiles: over the dead K and Q rows
  constexpr int kRtTerm = NT == 64 ? 16384 : 64;                // byte distance from the hi to the lo operand
  constexpr int kMtTerm = NT == 64 ? 8192 : 64;
  constexpr int kMtBytes = NT == 64 ? 16384 : 4096;
  static_assert(kCompact || (NT == 64 ? 32768 : 16384) <= LY::kRec, "right-hand-side tiles overflow the dump area");
  // byte offset of element (row, col) of operand term 0 (hi) or 1 (lo): with NT = 64 the lo operand is a tile of
  // its own `term_bytes` on, with NT = 32 it is the upper half (k bytes 64..127) of the same swizzled rows
  auto tile_off = [](int row, int col, int term, int term_bytes) {
    const int chunk = NT == 64 ? (col >> 3) : term * 4 + (col >> 3);
    return (NT == 64 ? term * term_bytes : 0) + (int)sw128_offset(row, chunk) + (col & 7) * 2;
  };
  // ---- A and W along each node's ancestry (sixteen lanes per node); meanwhile the M tiles are cleared ----
  for (int i = tid; i < kMtBytes / 16; i += kThreads)             // bounded: <= 4 rounds
    *reinterpret_cast<uint4*>(smem + kMt + i * 16) = make_uint4(0u, 0u, 0u, 0u);
  if (tid < 2) sm.bad[tid] = 0u;
  {
    const int j = tid & 15, ln = tid >> 4;
#pragma unroll
    for (int m = 0; m < NT / 16; ++m) {
      if (16 * m >= N) break;                                       // uniform
      const int pi = ln + 16 * m;
      const int meta = sm.meta[pi];
      const int D = pi < N ? ((meta >> 16) & 0xFF) : 0;             // depth, 1..16 (the same in all 16 lanes)
      const bool in = j < D;
      const int a = sm.anc[pi][j];                                  // 0 beyond the depth
      float incl = in ? sm.alpha[a] : 1.f;
#pragma unroll
      for (int off = 1; off < 16; off <<= 1) {
        const float v = __shfl_down_sync(0xffffffffu, incl, off, 16);
        if (j + off < 16) incl *= v;
      }
      float excl = __shfl_down_sync(0xffffffffu, incl, 1, 16);      // product over the lanes above j
      if (j == 15) excl = 1.f;
      const float g_t = __shfl_sync(0xffffffffu, incl, 0, 16);      // product over the whole path
      float ksa = 1.f;
      if (s.l2norm && in) ksa = rsqrtf(dump[a * LY::kStride + a] + s.l2_eps);
      const float ks_t = __shfl_sync(0xffffffffu, ksa, D > 0 ? D - 1 : 0, 16);
      const float qs_t = s.l2norm ? s.scale * rsqrtf(sm.qq[pi] + s.l2_eps) : s.scale;
      const float b_t = sm.beta[pi];
      float kk = 0.f, qk = 0.f;
      if (in) { kk = dump[pi * LY::kStride + a]; qk = dump[(NT + pi) * LY::kStride + a]; }
      Am[pi * 16 + j] = j < D - 1 ? b_t * excl * ks_t * ksa * kk : 0.f;   // no entry for the node itself
      Wm[pi * 16 + j] = in ? qs_t * excl * ksa * qk : 0.f;
      if (j == 0) {
        sm.qs[pi] = g_t * qs_t;                                     // factor of S0 q
        sm.ks[pi] = b_t * g_t * ks_t;                               // factor of S0 k
        sm.out_off[pi] = (pi < N && ((meta >> 24) & 1)) ? (uint32_t)((((size_t)b * s.Ns + (meta & 0xFFFF)) * s.Hv + hv) * kD) : 0xFFFFFFFFu;
      }
    }
  }
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");            // this thread's pieces of V
  tc_fence_before();                                                // the Gram columns were read: they take the product below
  __syncthreads();                                                  // A, W, V, cleared M tiles in place; the dump is dead
  // ---- M by back substitution (four lanes per node), scattered as bf16 hi + lo into the M tiles -----------
  if (tid < 4 * NT) {                                               // whole warps
    const int pi = tid >> 2, q4 = tid & 3;
    const int D = pi < N ? ((sm.meta[pi] >> 16) & 0xFF) : 0;
    float4 w = *reinterpret_cast<const float4*>(Wm + pi * 16 + 4 * q4);
    const int Dw = __reduce_max_sync(0xffffffffu, D);
    for (int jh = Dw - 1; jh >= 1; --jh) {                          // bounded: <= 15 steps
      const int e = jh & 3;
      const float cand = e == 0 ? w.x : e == 1 ? w.y : e == 2 ? w.z : w.w;
      const float mval = __shfl_sync(0xffffffffu, cand, (lane & ~3) | (jh >> 2));
      if (jh < D) {
        const float4 ar = *reinterpret_cast<const float4*>(Am + sm.anc[pi][jh] * 16 + 4 * q4);
        w.x = fmaf(-mval, ar.x, w.x); w.y = fmaf(-mval, ar.y, w.y);
        w.z = fmaf(-mval, ar.z, w.z); w.w = fmaf(-mval, ar.w, w.w);
      }
    }
    const uint32_t a4 = *reinterpret_cast<const uint32_t*>(&sm.anc[pi][4 * q4]);
    const float mv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (4 * q4 + e < D) {
        const int sidx = (a4 >> (8 * e)) & 0xFF;
        const __nv_bfloat16 h0 = __float2bfloat16_rn(mv[e]);
        const __nv_bfloat16 h1 = __float2bfloat16_rn(mv[e] - __bfloat162float(h0));
        *reinterpret_cast<__nv_bfloat16*>(smem + kMt + tile_off(pi, sidx, 0, kMtTerm)) = h0;
        *reinterpret_cast<__nv_bfloat16*>(smem + kMt + tile_off(pi, sidx, 1, kMtTerm)) = h1;
      }
    }
  }
  // ---- right-hand sides: lane = value row, each half of the CTA half of the nodes, eight nodes per 16-byte
  //      store; padding nodes are written as zeros (their V bytes are stale) ----------------------------------
  {
    constexpr int kPer = NT / 2;                                    // nodes per thread
    const int n0 = grp * kPer;
    uint32_t pk[kPer];
    tmem_ld16_issue(tmem_lane + n0, pk);
    if constexpr (kPer == 32) tmem_ld16_issue(tmem_lane + n0 + 16, pk + 16);
    tmem_ld_wait();
#pragma unroll
    for (int c = 0; c < kPer / 8; ++c) {
      const int s0 = n0 + 8 * c;
      const float4 b0 = *reinterpret_cast<const float4*>(&sm.beta[s0]), b1 = *reinterpret_cast<const float4*>(&sm.beta[s0 + 4]);
      const float4 c0 = *reinterpret_cast<const float4*>(&sm.ks[s0]), c1 = *reinterpret_cast<const float4*>(&sm.ks[s0 + 4]);
      const float bt[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
      const float ck[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
      float r8[8];
      uint32_t hi[4], lo[4];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int sn = s0 + e;
        const float v = __bfloat162float(Vs[sn * kD + vrow]);
        r8[e] = sn < N ? fmaf(bt[e], v, -ck[e] * __uint_as_float(pk[8 * c + e])) : 0.f;
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        __nv_bfloat162 h = __floats2bfloat162_rn(r8[2 * e], r8[2 * e + 1]);
        hi[e] = *reinterpret_cast<uint32_t*>(&h);
      }
      // inf or NaN among the eight (as rounded to bf16)?  One test on the OR of the words: an exponent field of all
      // ones shows as 0x7F80; the OR can show it where no single value has it, which only costs the exact look below
      if ((((hi[0] | hi[1] | hi[2] | hi[3]) & 0x7F807F80u) + 0x00800080u) & 0x80008000u) {      // rare
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          if (((hi[e >> 1] >> (16 * (e & 1))) & 0x7F80u) == 0x7F80u) {
            const int sn = s0 + e;
            atomicOr(&sm.bad[sn >> 5], 1u << (sn & 31));
            r8[e] = 0.f;
            hi[e >> 1] &= (e & 1) ? 0x0000FFFFu : 0xFFFF0000u;
          }
        }
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 hf = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&hi[e]));
        __nv_bfloat162 l = __floats2bfloat162_rn(r8[2 * e] - hf.x, r8[2 * e + 1] - hf.y);
        lo[e] = *reinterpret_cast<uint32_t*>(&l);
      }
      *reinterpret_cast<uint4*>(smem + kRt + tile_off(vrow, s0, 0, kRtTerm)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
      *reinterpret_cast<uint4*>(smem + kRt + tile_off(vrow, s0, 1, kRtTerm)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    }
  }
  fence_async_proxy();          // generic-proxy writes -> visible to the tensor core's async proxy
  __syncthreads();
  // ---- O = RHS M^T: hi.hi + hi.lo + lo.hi, NT / 16 contraction steps each ----------------------------------
  if (tid == 0) {
    tc_fence_after();
    constexpr uint32_t idesc = umma_idesc(128, NT);
    const uint64_t d_r = umma_desc(sbase + kRt), d_m = umma_desc(sbase + kMt);
    constexpr uint64_t r_lo = (uint64_t)(kRtTerm >> 4), m_lo = (uint64_t)(kMtTerm >> 4);
#pragma unroll
    for (int ks = 0; ks < NT / 16; ++ks) {
      const uint64_t koff = (uint64_t)((ks * 32) >> 4);
      umma(tmem + LY::kGramCol, d_r + koff, d_m + koff, idesc, ks ? 1u : 0u);
      umma(tmem + LY::kGramCol, d_r + koff, d_m + m_lo + koff, idesc, 1u);
      umma(tmem + LY::kGramCol, d_r + r_lo + koff, d_m + koff, idesc, 1u);
    }
    umma_commit(&sm.mbar);
  }
  const bool done = mbar_wait(&sm.mbar, phase);
  phase ^= 1;
  tc_fence_after();
  if (!done) return false;
  // ---- outputs: they leave tensor memory lane = value row, cross shared memory [node][row] (over the dead
  //      right-hand-side tiles) and are written one node per warp, 256 or 512 contiguous bytes at a time -----------
  float* stage = reinterpret_cast<float*>(smem + kRt);
  static_assert(kCompact || NT * kD * 4 <= LY::kRec, "output staging overflows the dump area");
  {
    constexpr int kPer = NT / 2;
    const int n0 = grp * kPer;
    uint32_t oo[kPer], pq[kPer];
    tmem_ld16_issue(tmem_lane + LY::kGramCol + n0, oo);
    tmem_ld16_issue(tmem_lane + NT + n0, pq);
    if constexpr (kPer == 32) {
      tmem_ld16_issue(tmem_lane + LY::kGramCol + n0 + 16, oo + 16);
      tmem_ld16_issue(tmem_lane + NT + n0 + 16, pq + 16);
    }
    tmem_ld_wait();
#pragma unroll
    for (int e4 = 0; e4 < kPer; e4 += 4) {
      const float4 cq4 = *reinterpret_cast<const float4*>(&sm.qs[n0 + e4]);
      const float cqs[4] = {cq4.x, cq4.y, cq4.z, cq4.w};
#pragma unroll
      for (int k = 0; k < 4; ++k)
        stage[(n0 + e4 + k) * kD + vrow] = fmaf(cqs[k], __uint_as_float(pq[e4 + k]), __uint_as_float(oo[e4 + k]));
    }
  }
  __syncthreads();
  const bool any_bad = (sm.bad[0] | sm.bad[1]) != 0u;               // uniform over the CTA; rare
  const int warp = tid >> 5;
  for (int pi = warp; pi < N; pi += kWarps) {                       // bounded: <= 8 rounds
    const uint32_t off = sm.out_off[pi];
    if (off == 0xFFFFFFFFu) continue;
    float4 o = *reinterpret_cast<const float4*>(stage + pi * kD + 4 * lane);
    if (any_bad) {
      const int D = (sm.meta[pi] >> 16) & 0xFF;
      bool hit = false;
      for (int j = 0; j < D; ++j) {                                 // bounded: <= 16
        const int a = sm.anc[pi][j];
        hit = hit || ((sm.bad[a >> 5] >> (a & 31)) & 1u);
      }
      if (hit) o = make_float4(__uint_as_float(0x7FC00000u), __uint_as_float(0x7FC00000u), __uint_as_float(0x7FC00000u), __uint_as_float(0x7FC00000u));
    }
    if (s.out_dtype == LUMO_BF16) {
      __nv_bfloat162 b01 = __floats2bfloat162_rn(o.x, o.y), b23 = __floats2bfloat162_rn(o.z, o.w);
      *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(L.out) + (size_t)off + 4 * lane) =
          make_uint2(*reinterpret_cast<uint32_t*>(&b01), *reinterpret_cast<uint32_t*>(&b23));
    } else {
      *reinterpret_cast<float4*>(reinterpret_cast<float*>(L.out) + (size_t)off + 4 * lane) = o;
    }
  }
  return true;
}

// NT = node tile of the MMAs: 64, or 32 when no group of the launch has more than 32 nodes (K rows
// 0..NT-1 and Q rows NT..2NT-1 of the operand tile; the products occupy NT + NT + NT columns)
// kFused: before anything else the previous cycle's accepted path is replayed into the state rows as
// they pass through the registers (same per-token update as the commit kernel), and the rows are
// written back in place; the scan then runs from the updated state.  One group per sequence only.
// kDirect: the triangular system is solved on scalars per node (M = W (I + A)^-1 along each ancestry, no
// dependency between nodes) and every output is one pass over its path; no level-by-level substitution.
// kTensor (with kDirect): the output sum of the closed form runs on the tensor core (direct_tail_tc).
template <int NT, bool kFused, bool kCompact = false, bool kDirect = false, bool kTensor = false>
__device__ __forceinline__ void scan_gram_body(const Shape& s, const TreeDev& t, const LayerBatch& lb, int n_items,
                                               const FusedPrev* fp) {
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment for the swizzled operand tiles; plain pointer arithmetic on the shared
  // array keeps the pointers in the shared address space
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  static_assert(!kCompact || (NT == 32 && !kFused), "the compact layout serves the 32-node tile of the plain scan");
  using LY = GL<kCompact>;
  Small& sm = *reinterpret_cast<Small*>(smem + LY::kSmall);
  float* dump = reinterpret_cast<float*>(smem + kOffDump);
  float* dls = reinterpret_cast<float*>(smem + kOffDump);     // [nodes + 1][128]; the last row stays zero
  float* Pq = reinterpret_cast<float*>(smem + LY::kKQ);
  NodeRec* recs = reinterpret_cast<NodeRec*>(smem + LY::kRec);
  const __nv_bfloat16* Vs = reinterpret_cast<const __nv_bfloat16*>(smem + LY::kV);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int grp = tid >> 7;            // half of the CTA: 0 or 1
  const int vrow = tid & 127;          // value row = TMEM lane
  const int rep = s.Hv / s.Hk;

  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&sm.tmem_base)), "r"(LY::kTmem) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  if (tid == 0) { mbar_init(&sm.mbar, 1); sm.timed_out = 0; }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  const uint32_t tmem_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16);   // this warp's 32 lanes
  uint32_t phase = 0;
  // compact mode: state rows of this thread r = 16 u + 2 warp + (lane >> 4), four floats at column
  // 4 (lane & 15) of the current 64-column half
  const int srow0 = 2 * warp + (lane >> 4), c4 = lane & 15;
  const uint32_t s0_off0 = sw128_offset(srow0, c4 >> 1) + (c4 & 1) * 8;   // rows 16 u on: + 2048 u

  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {   // bounded: n_items
    const int hv = item % s.Hv;
    const int gi = (item / s.Hv) % t.n_groups;                     // node group
    const int layer = item / (s.Hv * t.n_groups);
    // A tree of one group (every tree when there are as many groups as sequences) needs no look-up: group =
    // sequence, all nodes, first group.  That takes one dependent load off the head of the item's chain
    // (group -> state row -> state).
    const bool one_group = t.n_groups == s.B;
    int4 ginfo = make_int4(gi, s.N, 1, 0);
    if (!one_group) ginfo = *reinterpret_cast<const int4*>(t.tc_group + gi * 4);
    const int b = ginfo.x, N = ginfo.y;                            // sequence, nodes in this group
    const bool first_group = ginfo.z != 0;                         // writes the per-sequence zero rows
    const LayerPtrs& L = lb.l[layer];
    const int g = hv / rep;
    const int row = L.state_row[b];
    const size_t out_row_stride = (size_t)s.Hv * kD;
    // The item this CTA takes next: its state and operand rows are pulled into L2 while this item
    // computes (requests issued behind the dependency wait below), so that its own loads find them there.
    const int nxt = item + (int)gridDim.x;
    // (trees cut into several groups re-read one state per group from L2 anyway: there it measured slower)
    const bool has_next = !kFused && nxt < n_items && t.n_groups == s.B;
    int n_hv = 0, n_layer = 0, n_b = 0, n_meta = -1, n_row = -1;
    if (has_next) {
      n_hv = nxt % s.Hv;
      const int n_gi = (nxt / s.Hv) % t.n_groups;
      n_layer = nxt / (s.Hv * t.n_groups);
      const int4 gi4 = one_group ? make_int4(n_gi, s.N, 1, 0) : *reinterpret_cast<const int4*>(t.tc_group + n_gi * 4);
      n_b = gi4.x;
      if (tid < gi4.y) n_meta = t.tc_meta[n_gi * kNT + tid];
      n_row = lb.l[n_layer].state_row[n_b];
    }

    if (row < 0 || row >= s.n_state_rows) {   // skipped sequence: zero outputs
      pdl_wait();                             // every path through the kernel passes its dependency wait
      if (first_group) {
        for (int ps = grp; ps < s.Ns; ps += 2)
          store_out(L.out, ((size_t)b * s.Ns + ps) * out_row_stride + hv * kD + vrow, s.out_dtype, 0.f);
        if (L.status && hv == 0 && tid == 0) L.status[b] = row < 0 ? LUMO_SEQ_OK : LUMO_SEQ_BAD_ROW;
        if constexpr (kFused) {
          int32_t* pst = fp->lb.l[layer].status;
          if (pst && hv == 0 && tid == 0) pst[b] = row < 0 ? LUMO_SEQ_OK : LUMO_SEQ_BAD_ROW;
        }
      }
      continue;
    }
    if (first_group && L.status && hv == 0 && tid == 0) L.status[b] = LUMO_SEQ_OK;
    int plen = 0;
    if constexpr (kFused) {
      // the accepted path of the previous cycle: entries, parents, physical rows (one level of dependent loads)
      PrevStage& ps = *reinterpret_cast<PrevStage*>(smem + kOffPrev);
      plen = fp->len[b];
      const int lcap = plen < 0 ? 0 : (plen > fp->lmax ? 0 : plen);
      if (tid >= 2 * kNT + 32 && tid < 2 * kNT + 32 + lcap) {
        const int tt = tid - (2 * kNT + 32);
        const int a = fp->accepted[(size_t)b * fp->lmax + tt];
        const bool ok = a >= 0 && a < fp->N;
        ps.acc[tt] = a;
        ps.par[tt] = ok ? fp->parent[(size_t)b * fp->N + a] : -2;
        ps.phys[tt] = ok ? fp->slot[(size_t)b * fp->N + a] : 0;
      }
    }
    // The pre-tree state is not written by the kernel before this one and its address needs no
    // table: its first half (warp w takes rows w, w+8, ...; one 512-byte row per instruction) is
    // requested first of all, ahead of the table loads and of the dependency wait.
    const float* S0 = L.state + ((size_t)row * s.Hv + hv) * kD * kD;
    float4 x[8];
#pragma unroll
    for (int u = 0; u < 8; ++u)
      x[u] = kCompact ? *reinterpret_cast<const float4*>(S0 + (size_t)(16 * u + srow0) * kD + 4 * c4)
                      : *reinterpret_cast<const float4*>(S0 + (size_t)(warp + 8 * u) * kD + lane * 4);
    // ---- a. per-node tables (the addresses of everything else depend on them) -------------------
    if (tid < kNT) {
      sm.meta[tid] = tid < N ? t.tc_meta[gi * kNT + tid] : 0;
    } else if (tid < 2 * kNT) {
      const int pi = tid - kNT;
      uint4 av = make_uint4(0, 0, 0, 0);
      if (pi < N) av = *reinterpret_cast<const uint4*>(t.tc_anc + ((size_t)gi * kNT + pi) * 16);
      *reinterpret_cast<uint4*>(sm.anc[pi]) = av;
    } else if (tid < 2 * kNT + 20) {
      sm.lvl[tid - 2 * kNT] = t.tc_lvl[gi * 20 + tid - 2 * kNT];
    }
    bool replay = false;
    __syncthreads();
    if constexpr (kFused) {
      PrevStage& ps = *reinterpret_cast<PrevStage*>(smem + kOffPrev);
      const LayerPtrs& PL = fp->lb.l[layer];
      const int st = check_path_staged(ps.acc, ps.par, fp->N, plen, fp->lmax);    // same answer in every thread
      if (PL.status && hv == 0 && tid == 0) PL.status[b] = st;
      replay = st == LUMO_SEQ_OK && plen > 0;
      if (replay) {
        // recorded key and value rows of the accepted nodes, gates; these were complete long before
        // this kernel's predecessor started
        const __nv_bfloat16* pk = reinterpret_cast<const __nv_bfloat16*>(PL.k);
        const __nv_bfloat16* pv = reinterpret_cast<const __nv_bfloat16*>(PL.v);
        for (int e = tid; e < plen * 32; e += kThreads) {            // bounded: <= 512
          const int tt = e >> 5, c = e & 15;
          const size_t pr = (size_t)b * fp->Ns + ps.phys[tt];
          if ((e & 16) == 0)
            *reinterpret_cast<uint4*>(&ps.k[tt][c * 8]) = *reinterpret_cast<const uint4*>(pk + (pr * s.Hk + g) * kD + c * 8);
          else
            *reinterpret_cast<uint4*>(&ps.v[tt][c * 8]) = *reinterpret_cast<const uint4*>(pv + (pr * s.Hv + hv) * kD + c * 8);
        }
        if (tid < plen) ps.gates[tid] = load_gates(PL, s, ((size_t)b * fp->Ns + ps.phys[tid]) * s.Hv + hv, hv);
      }
      __syncthreads();
      if (replay) {
        for (int tt = warp; tt < plen; tt += kWarps) {               // bounded: <= 16
          const uint2 w = *reinterpret_cast<const uint2*>(&ps.k[tt][4 * lane]);
          const float k0 = __uint_as_float(w.x << 16), k1 = __uint_as_float(w.x & 0xFFFF0000u);
          const float k2 = __uint_as_float(w.y << 16), k3 = __uint_as_float(w.y & 0xFFFF0000u);
          float kk = fmaf(k0, k0, fmaf(k1, k1, fmaf(k2, k2, k3 * k3)));
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) kk += __shfl_xor_sync(0xffffffffu, kk, o);
          if (lane == 0) ps.ks[tt] = s.l2norm ? rsqrtf(kk + s.l2_eps) : 1.f;
        }
      }
      __syncthreads();
    }
    // ---- b. gates (consumed much later); K and Q rows -> swizzled operand tile (cp.async) ---------
    // K, Q, V may still be in the making (the convolution runs right before this kernel): everything
    // above touched only the descriptor tables and the state.  The dependent kernel (commit) is let in
    // afterwards: it reads freely and writes only behind its own wait.
    pdl_wait();
    // A fused launch rewrites the state, which a dependent (a commit, the next scan) requests ahead of
    // its own wait: it lets nobody in before it has finished.
    if constexpr (!kFused) pdl_trigger();
    if (has_next) {
      if (n_meta >= 0) {      // a node's key, query and value rows (256 bytes = two lines each) and its gates
        const LayerPtrs& NL = lb.l[n_layer];
        const size_t pr = (size_t)n_b * s.Ns + (n_meta & 0xFFFF);
        const int n_g = n_hv / rep;
        const __nv_bfloat16* pk = reinterpret_cast<const __nv_bfloat16*>(NL.k) + (pr * s.Hk + n_g) * kD;
        const __nv_bfloat16* pq = reinterpret_cast<const __nv_bfloat16*>(NL.q) + (pr * s.Hk + n_g) * kD;
        const __nv_bfloat16* pv = reinterpret_cast<const __nv_bfloat16*>(NL.v) + (pr * s.Hv + n_hv) * kD;
        prefetch_l2(pk); prefetch_l2(pk + 64);
        prefetch_l2(pq); prefetch_l2(pq + 64);
        prefetch_l2(pv); prefetch_l2(pv + 64);
        const size_t gsz = s.gate_dtype == LUMO_BF16 ? 2 : 4;
        prefetch_l2(reinterpret_cast<const unsigned char*>(NL.alpha) + (pr * s.Hv + n_hv) * gsz);
        prefetch_l2(reinterpret_cast<const unsigned char*>(NL.beta) + (pr * s.Hv + n_hv) * gsz);
      }
      if (n_row >= 0 && n_row < s.n_state_rows) {      // the state: 64 KiB = 512 lines, two per thread
        const float* ns0 = lb.l[n_layer].state + ((size_t)n_row * s.Hv + n_hv) * kD * kD;
        prefetch_l2(ns0 + 32 * tid);
        prefetch_l2(ns0 + 32 * (tid + kThreads));
      }
    }
    if constexpr (kFused) {
      // The convolution before this kernel read the committed history through the path; now that it has
      // finished, the history buffer itself is brought up to date: the value heads of a sequence share
      // out the channels, a thread moves its 16 bytes of all three rows (reads before writes).
      if (fp->hist_in_kernels && replay && warp == kWarps - 1) {
        const PrevStage& ps = *reinterpret_cast<const PrevStage*>(smem + kOffPrev);
        const LayerPtrs& PL = fp->lb.l[layer];
        const int chunks = s.C / 8;                                    // 16-byte pieces of a row of bf16 channels
        const int per_head = (chunks + s.Hv - 1) / s.Hv;
        __nv_bfloat16* hist = reinterpret_cast<__nv_bfloat16*>(L.conv_hist) + (size_t)row * 3 * s.C;
        const __nv_bfloat16* xprev = reinterpret_cast<const __nv_bfloat16*>(PL.x) + (size_t)b * fp->Ns * s.C;
        for (int c = hv * per_head + lane; c < min(chunks, (hv + 1) * per_head); c += 32) {   // bounded: per_head
          uint4 rows3[3];
#pragma unroll
          for (int j = 0; j < 3; ++j) {
            const int q = plen + j;    // index into [old0 old1 old2 x_a0 x_a1 ...]
            const __nv_bfloat16* src = q < 3 ? hist + (size_t)q * s.C : xprev + (size_t)ps.phys[q - 3] * s.C;
            rows3[j] = *reinterpret_cast<const uint4*>(src + c * 8);
          }
#pragma unroll
          for (int j = 0; j < 3; ++j) *reinterpret_cast<uint4*>(hist + (size_t)j * s.C + c * 8) = rows3[j];
        }
      }
    }
    float gate_a = 1.f, gate_b = 0.f;
    if (tid < N) {
      const size_t pr = (size_t)b * s.Ns + (sm.meta[tid] & 0xFFFF);
      const float2 gates = load_gates(L, s, pr * s.Hv + hv, hv);
      gate_a = gates.x;
      gate_b = gates.y;
    }
    {
      const __nv_bfloat16* kg = reinterpret_cast<const __nv_bfloat16*>(L.k);
      const __nv_bfloat16* qg = reinterpret_cast<const __nv_bfloat16*>(L.q);
      constexpr int kCopies = 2 * NT * 16 / kThreads;   // 16-byte pieces of the 2 NT rows, per thread
      const __nv_bfloat16* src[kCopies];
#pragma unroll
      for (int i = 0; i < kCopies; ++i) {                // addresses first, so that the copies issue back to back
        const int idx = i * kThreads + tid;
        const int R = idx >> 4, c = idx & 15;
        const int pi = R & (NT - 1);
        const size_t pr = (size_t)b * s.Ns + (sm.meta[pi] & 0xFFFF);
        src[i] = pi < N ? (R < NT ? kg : qg) + (pr * s.Hk + g) * kD + c * 8 : nullptr;
      }
#pragma unroll
      for (int i = 0; i < kCopies; ++i) {
        const int idx = i * kThreads + tid;
        const int R = idx >> 4, c = idx & 15;
        const uint32_t dst = sbase + LY::kKQ + (c >> 3) * 16384 + sw128_offset(R, c & 7);
        if (src[i]) cp_async16(dst, src[i]);
        else asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};\n" ::"r"(dst), "r"(0u) : "memory");
      }
      asm volatile("cp.async.commit_group;\n" ::: "memory");
    }
    // ---- c. pre-tree state -> bf16 hi + lo operand tiles ------------------------------------------
    {
      const int kblock = lane >> 4, chunk = (lane & 15) >> 1, half = lane & 1;
      // fused mode: rows r0 + 8u of the state, held as x[u], take the accepted path's updates
      // (u_r = S_r . k, delta_r = beta (v_r - alpha ks u_r), S_r <- alpha S_r + delta_r ks k) and go back to memory
      auto replay_rows = [&](int r0) {
        if constexpr (kFused) {
          if (!replay) return;
          const PrevStage& ps = *reinterpret_cast<const PrevStage*>(smem + kOffPrev);
          for (int tt = 0; tt < plen; ++tt) {                        // bounded: <= 16
            const uint2 w = *reinterpret_cast<const uint2*>(&ps.k[tt][4 * lane]);
            const float4 kv = make_float4(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xFFFF0000u),
                                          __uint_as_float(w.y << 16), __uint_as_float(w.y & 0xFFFF0000u));
            const float a = ps.gates[tt].x, bt = ps.gates[tt].y, ks = ps.ks[tt];
            float p[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) p[u] = fmaf(x[u].x, kv.x, fmaf(x[u].y, kv.y, fmaf(x[u].z, kv.z, x[u].w * kv.w)));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
#pragma unroll
              for (int u = 0; u < 8; ++u) p[u] += __shfl_xor_sync(0xffffffffu, p[u], o);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const float vv = __bfloat162float(ps.v[tt][r0 + 8 * u]);
              const float gk = bt * (vv - a * (ks * p[u])) * ks;
              x[u].x = fmaf(a, x[u].x, gk * kv.x); x[u].y = fmaf(a, x[u].y, gk * kv.y);
              x[u].z = fmaf(a, x[u].z, gk * kv.z); x[u].w = fmaf(a, x[u].w, gk * kv.w);
            }
          }
          float* Sw = const_cast<float*>(S0);
#pragma unroll
          for (int u = 0; u < 8; ++u) *reinterpret_cast<float4*>(Sw + (size_t)(r0 + 8 * u) * kD + lane * 4) = x[u];
        }
      };
      if constexpr (kCompact) {
        // first 64-column half -> tiles; the second half is requested at once and converted after the
        // products of the first
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          split_store<LY::kAhi, LY::kAlo>(smem, s0_off0 + 2048 * u, x[u]);
          x[u] = *reinterpret_cast<const float4*>(S0 + (size_t)(16 * u + srow0) * kD + 64 + 4 * c4);
        }
      } else {
        replay_rows(warp);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          split_store(smem, kblock * 16384 + sw128_offset(warp + 8 * u, chunk) + half * 8, x[u]);
          x[u] = *reinterpret_cast<const float4*>(S0 + (size_t)(warp + 8 * (8 + u)) * kD + lane * 4);   // second half
        }
        replay_rows(warp + 64);
#pragma unroll
        for (int u = 0; u < 8; ++u)
          split_store(smem, kblock * 16384 + sw128_offset(warp + 8 * (8 + u), chunk) + half * 8, x[u]);
      }
    }
    if (tid < kNT) { sm.alpha[tid] = gate_a; sm.beta[tid] = gate_b; }
    // padding rows: zero outputs
    if (first_group && s.Ns > s.N)
      for (int ps = grp; ps < s.Ns; ps += 2)
        if (t.slot_inv[b * s.Ns + ps] < 0)
          store_out(L.out, ((size_t)b * s.Ns + ps) * out_row_stride + hv * kD + vrow, s.out_dtype, 0.f);
    asm volatile("cp.async.wait_group 0;\n" ::: "memory");
    fence_async_proxy();          // generic-proxy writes -> visible to the tensor core's async proxy
    __syncthreads();
    // ---- e. MMAs: Gram = [K;Q] K^T, P = S0 [K|Q]^T (hi + lo); meanwhile |q|^2 when normalising ----
    if (tid == 0) {
      tc_fence_after();
      constexpr uint32_t idesc_p = umma_idesc(128, 2 * NT), idesc_g = umma_idesc(128, NT);
      const uint64_t d_kq = umma_desc(sbase + LY::kKQ), d_hi = umma_desc(sbase + LY::kAhi), d_lo = umma_desc(sbase + LY::kAlo);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const uint64_t koff = (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
        umma(tmem + LY::kGramCol, d_kq + koff, d_kq + koff, idesc_g, ks ? 1u : 0u);
      }
      if constexpr (kCompact) {
        // the state tiles hold the first 64-column half only: its four contraction steps now
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          const uint64_t koff = (uint64_t)((ks * 32) >> 4);
          umma(tmem, d_hi + koff, d_kq + koff, idesc_p, ks ? 1u : 0u);
          umma(tmem, d_lo + koff, d_kq + koff, idesc_p, 1u);
        }
      } else {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t koff = (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
          umma(tmem, d_hi + koff, d_kq + koff, idesc_p, ks ? 1u : 0u);
        }
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t koff = (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
          umma(tmem, d_lo + koff, d_kq + koff, idesc_p, 1u);
        }
      }
      umma_commit(&sm.mbar);
    } else if (grp == 1 && s.l2norm && vrow < NT) {
      const int R = NT + vrow;   // tile row of q_vrow (the tensor core only reads the tile)
      float qq = 0.f;
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const uint4 w = *reinterpret_cast<const uint4*>(smem + LY::kKQ + (c >> 3) * 16384 + sw128_offset(R, c & 7));
        const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float lo = __uint_as_float(ws[e] << 16), hi = __uint_as_float(ws[e] & 0xFFFF0000u);
          qq = fmaf(lo, lo, qq); qq = fmaf(hi, hi, qq);
        }
      }
      sm.qq[vrow] = qq;
    }
    // ---- f. wait for the tensor core (bounded) ---------------------------------------------------
    if (!mbar_wait(&sm.mbar, phase)) sm.timed_out = 1;
    phase ^= 1;
    tc_fence_after();
    __syncthreads();
    if (sm.timed_out) {    // give up on this and all further items; report, free TMEM, leave
      if (L.status && tid == 0) L.status[b] = LUMO_SEQ_TIMEOUT;
      break;
    }
    if constexpr (kCompact) {
      // second 64-column half of the state through the same tiles, accumulated onto the first
#pragma unroll
      for (int u = 0; u < 8; ++u) split_store<LY::kAhi, LY::kAlo>(smem, s0_off0 + 2048 * u, x[u]);
      fence_async_proxy();
      __syncthreads();
      if (tid == 0) {
        tc_fence_after();
        constexpr uint32_t idesc_p = umma_idesc(128, 2 * NT);
        const uint64_t d_kq = umma_desc(sbase + LY::kKQ + 16384), d_hi = umma_desc(sbase + LY::kAhi), d_lo = umma_desc(sbase + LY::kAlo);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          const uint64_t koff = (uint64_t)((ks * 32) >> 4);
          umma(tmem, d_hi + koff, d_kq + koff, idesc_p, 1u);
          umma(tmem, d_lo + koff, d_kq + koff, idesc_p, 1u);
        }
        umma_commit(&sm.mbar);
      }
      if (!mbar_wait(&sm.mbar, phase)) sm.timed_out = 1;
      phase ^= 1;
      tc_fence_after();
      __syncthreads();
      if (sm.timed_out) {
        if (L.status && tid == 0) L.status[b] = LUMO_SEQ_TIMEOUT;
        break;
      }
    }
    // ---- g. V rows -> shared (space of the dead S0 tiles); Gram rows out of tensor memory ----------
    {
      const __nv_bfloat16* vg = reinterpret_cast<const __nv_bfloat16*>(L.v);
#pragma unroll
      for (int i = 0; i < NT * 16 / kThreads; ++i) {
        const int idx = i * kThreads + tid;
        const int pi = idx >> 4, c = idx & 15;
        if (pi < N) {
          const size_t pr = (size_t)b * s.Ns + (sm.meta[pi] & 0xFFFF);
          cp_async16(sbase + LY::kV + pi * 256 + c * 16, vg + (pr * s.Hv + hv) * kD + c * 8);
        }
      }
      asm volatile("cp.async.commit_group;\n" ::: "memory");
    }
    // both halves of the CTA read the Gram rows: 32 of the NT columns each (one half is enough for NT = 32)
    if (grp * 32 < NT) tmem_cols32_to_smem(tmem_lane + LY::kGramCol + grp * 32, dump + vrow * LY::kStride + grp * 32, 1);
    __syncthreads();
    if constexpr (kDirect && kTensor) {
      if (!direct_tail_tc<NT, LY, kCompact>(s, L, sm, smem, sbase, dump, Vs, tmem, tmem_lane, N, b, hv, tid, phase)) sm.timed_out = 1;
      tc_fence_before();
      __syncthreads();      // tensor memory and the aliased shared memory are free for the next item
      if (sm.timed_out) {
        if (L.status && tid == 0) L.status[b] = LUMO_SEQ_TIMEOUT;
        break;
      }
      continue;
    } else if constexpr (kDirect) {
      direct_tail<NT, LY>(s, L, sm, smem, dump, Vs, tmem_lane, N, b, hv, tid);
      tc_fence_before();
      __syncthreads();      // tensor memory and the aliased shared memory are free for the next item
      continue;
    }
    // ---- h. normalisation factors ------------------------------------------------------------------
    if (tid < NT) sm.ks[tid] = s.l2norm ? rsqrtf(dump[tid * LY::kStride + tid] + s.l2_eps) : 1.f;
    else if (tid < 2 * NT) sm.qs[tid - NT] = s.l2norm ? s.scale * rsqrtf(sm.qq[tid - NT] + s.l2_eps) : s.scale;
    __syncthreads();
    // ---- i. first half of the CTA: node records, one thread per (node, table); second half: the
    //         S0 q^ products move from tensor memory to shared memory [node][row] ---------------------
    if (grp == 0) {
      if (tid < 2 * NT) {
      const bool is_q = tid >= NT;
      const int pi = tid & (NT - 1);
      NodeRec& rec = recs[pi];
      const int meta = sm.meta[pi];
      const int D = pi < N ? ((meta >> 16) & 0xFF) : 0;          // depth, 1..16
      const float a_t = sm.alpha[pi], b_t = sm.beta[pi];
      const float self = is_q ? sm.qs[pi] : -b_t * sm.ks[pi];    // factor of the node itself (k side negated)
      const float* grow = dump + (is_q ? NT + pi : pi) * LY::kStride;
      float G = a_t;
      float w[16];
      uint32_t ao[8];
#pragma unroll
      for (int j = 15; j >= 0; --j) {                            // bounded: 16 depth slots
        float val = 0.f;
        uint32_t off = LY::kZero;
        if (j <= D - 2) {
          const int sidx = sm.anc[pi][j];
          val = self * G * sm.ks[sidx] * grow[sidx];
          G *= sm.alpha[sidx];
          off = sidx * kD;
        }
        w[j] = val;
        if (j & 1) ao[j >> 1] = off << 16; else ao[j >> 1] |= off;
      }
      float4* wdst = reinterpret_cast<float4*>(is_q ? rec.wq : rec.wk);
#pragma unroll
      for (int e = 0; e < 4; ++e) wdst[e] = make_float4(w[4 * e], w[4 * e + 1], w[4 * e + 2], w[4 * e + 3]);
      if (is_q) {
        rec.c0q = self * G;
        rec.wself = self * sm.ks[pi] * grow[pi];                 // k^_t . q^_t (G = 1)
        // a prefix node that another group emits is computed here but not written
        rec.out_off = ((meta >> 24) & 1) ? (uint32_t)((((size_t)b * s.Ns + (meta & 0xFFFF)) * s.Hv + hv) * kD) : 0xFFFFFFFFu;
      } else {
        rec.c0k = self * G;                                      // -beta_t g_t |k scale|
        rec.beta = b_t;
        uint4* adst = reinterpret_cast<uint4*>(rec.aoff);
        adst[0] = make_uint4(ao[0], ao[1], ao[2], ao[3]);
        adst[1] = make_uint4(ao[4], ao[5], ao[6], ao[7]);
      }
      }
    } else {
      for (int cb = 0; cb < (N + 31) / 32; ++cb)                 // bounded: <= 2
        tmem_cols32_to_smem(tmem_lane + NT + cb * 32, Pq + (cb * 32) * kD + vrow, kD);
    }
    asm volatile("cp.async.wait_group 0;\n" ::: "memory");
    __syncthreads();      // records, V and Pq are in place; the Gram dump is dead from here on
    // the S0 k^ products take the place of the dump; each delta later overwrites its own product
    if (grp * 32 < N) tmem_cols32_to_smem(tmem_lane + grp * 32, dls + (grp * 32) * kD + vrow, kD);
    if (tid < kD) dls[LY::kZero + tid] = 0.f;
    __syncthreads();
    // ---- j. forward substitution, level by level; one warp per node, lane l carries value rows
    //         4l .. 4l+3.  A node's record, v and S0 products are loaded before the barrier that
    //         publishes the previous level; only the ancestors' deltas are fetched after it ----------
    {
      auto load_ops = [&](NodeOps& op, int pi) {
        const NodeRec& rec = recs[pi];
        op.m = *reinterpret_cast<const float4*>(&rec.c0k);
        op.out_off = rec.out_off;
        op.vb = *reinterpret_cast<const uint2*>(Vs + pi * kD + 4 * lane);
        op.pk = *reinterpret_cast<const float4*>(dls + pi * kD + 4 * lane);
        op.pq = *reinterpret_cast<const float4*>(Pq + pi * kD + 4 * lane);
        op.ck = *reinterpret_cast<const float4*>(rec.wk);
        op.cq = *reinterpret_cast<const float4*>(rec.wq);
        op.ao = *reinterpret_cast<const uint2*>(rec.aoff);
      };
      // packed fp32 FMAs (two correctly rounded fp32 lanes per instruction: same bits as scalar fmaf)
      auto block4 = [&](float4& acc, float4& o, const float4& ck, const float4& cq, const uint2& ao) {
        const float4 d0 = *reinterpret_cast<const float4*>(dls + (ao.x & 0xFFFFu) + 4 * lane);
        const float4 d1 = *reinterpret_cast<const float4*>(dls + (ao.x >> 16) + 4 * lane);
        const float4 d2 = *reinterpret_cast<const float4*>(dls + (ao.y & 0xFFFFu) + 4 * lane);
        const float4 d3 = *reinterpret_cast<const float4*>(dls + (ao.y >> 16) + 4 * lane);
        float2 a01 = make_float2(acc.x, acc.y), a23 = make_float2(acc.z, acc.w);
        float2 o01 = make_float2(o.x, o.y), o23 = make_float2(o.z, o.w);
        auto step = [&](float k, float q, const float4& dd) {
          const float2 kk = make_float2(k, k), qq = make_float2(q, q);
          const float2 lo2 = make_float2(dd.x, dd.y), hi2 = make_float2(dd.z, dd.w);
          a01 = __ffma2_rn(kk, lo2, a01); a23 = __ffma2_rn(kk, hi2, a23);
          o01 = __ffma2_rn(qq, lo2, o01); o23 = __ffma2_rn(qq, hi2, o23);
        };
        step(ck.x, cq.x, d0);
        step(ck.y, cq.y, d1);
        step(ck.z, cq.z, d2);
        step(ck.w, cq.w, d3);
        acc = make_float4(a01.x, a01.y, a23.x, a23.y);
        o = make_float4(o01.x, o01.y, o23.x, o23.y);
      };
      const int lvl_lane = sm.lvl[lane < 20 ? lane : 19];          // lane d holds lvl[d]
      NodeOps op;
      int lo = 0;
      if (warp < __shfl_sync(0xffffffffu, lvl_lane, 1)) load_ops(op, warp);
      for (int d = 1; d <= 16; ++d) {                              // bounded: 16 levels
        const int hi = __shfl_sync(0xffffffffu, lvl_lane, d);      // nodes of depth d: [lo, hi)
        const int nblk = (d + 2) >> 2;                             // blocks of four ancestors
        for (int pi = lo + warp; pi < hi; pi += kWarps) {          // bounded: <= 64
          if (pi != lo + warp) load_ops(op, pi);
          const float c0k = op.m.x, beta = op.m.y, c0q = op.m.z, wself = op.m.w;
          float4 acc, o;
          acc.x = fmaf(beta, __uint_as_float(op.vb.x << 16), c0k * op.pk.x);
          acc.y = fmaf(beta, __uint_as_float(op.vb.x & 0xFFFF0000u), c0k * op.pk.y);
          acc.z = fmaf(beta, __uint_as_float(op.vb.y << 16), c0k * op.pk.z);
          acc.w = fmaf(beta, __uint_as_float(op.vb.y & 0xFFFF0000u), c0k * op.pk.w);
          o.x = c0q * op.pq.x; o.y = c0q * op.pq.y; o.z = c0q * op.pq.z; o.w = c0q * op.pq.w;
          if (d > 1) block4(acc, o, op.ck, op.cq, op.ao);          // uniform over the CTA
          for (int blk = 1; blk < nblk; ++blk) {                   // bounded: <= 3 more blocks
            const NodeRec& rec = recs[pi];
            block4(acc, o, *reinterpret_cast<const float4*>(rec.wk + 4 * blk), *reinterpret_cast<const float4*>(rec.wq + 4 * blk),
                   *reinterpret_cast<const uint2*>(rec.aoff + 4 * blk));
          }
          *reinterpret_cast<float4*>(dls + pi * kD + 4 * lane) = acc;           // delta of this node
          o.x = fmaf(wself, acc.x, o.x); o.y = fmaf(wself, acc.y, o.y);
          o.z = fmaf(wself, acc.z, o.z); o.w = fmaf(wself, acc.w, o.w);
          const size_t oi = (size_t)op.out_off + 4 * lane;
          if (op.out_off == 0xFFFFFFFFu) {
          } else if (s.out_dtype == LUMO_BF16) {
            __nv_bfloat162 o01 = __floats2bfloat162_rn(o.x, o.y), o23 = __floats2bfloat162_rn(o.z, o.w);
            *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(L.out) + oi) =
                make_uint2(*reinterpret_cast<uint32_t*>(&o01), *reinterpret_cast<uint32_t*>(&o23));
          } else {
            *reinterpret_cast<float4*>(reinterpret_cast<float*>(L.out) + oi) = o;
          }
        }
        lo = hi;
        if (lo >= N) break;                                        // uniform
        if (lo + warp < __shfl_sync(0xffffffffu, lvl_lane, d + 1)) load_ops(op, lo + warp);   // next level's first node
        __syncthreads();                                           // deltas of this level visible to the next
      }
    }
    tc_fence_before();
    __syncthreads();      // tensor memory and the aliased shared memory are free for the next item
  }

  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(LY::kTmem) : "memory");
}

template <int NT, bool kDirect, bool kTensor = false>
__global__ void __launch_bounds__(kThreads, 2)
scan_gram_kernel(Shape s, TreeDev t, LayerBatch lb, int n_items) {
  scan_gram_body<NT, false, false, kDirect, kTensor>(s, t, lb, n_items, nullptr);
}

// trees of at most 32 nodes, launches of several waves: three smaller CTAs per SM
template <bool kDirect, bool kTensor = false>
__global__ void __launch_bounds__(kThreads, 3)
scan_gram_compact_kernel(Shape s, TreeDev t, LayerBatch lb, int n_items) {
  scan_gram_body<32, false, true, kDirect, kTensor>(s, t, lb, n_items, nullptr);
}

template <int NT, bool kDirect, bool kTensor = false>
__global__ void __launch_bounds__(kThreads, 2)
scan_gram_fused_kernel(Shape s, TreeDev t, LayerBatch lb, int n_items, FusedPrev fp) {
  scan_gram_body<NT, true, false, kDirect, kTensor>(s, t, lb, n_items, &fp);
}

template <class K>
cudaError_t allow_smem(K kernel, int bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

}  // namespace

bool gram_supported(const Shape& s, int max_depth) {
  return s.d == kD && s.in_dtype == LUMO_BF16 && s.snapshot_mode == 0 && max_depth <= 16;
}

cudaError_t launch_scan_gram(const Shape& s, const TreeDev& t, const LayerBatch& lb, int sm_count, bool pdl, int tail,
                             cudaStream_t st) {
  const bool direct = tail != 0;
  const int items = s.n_layers * t.n_groups * s.Hv;
  static bool configured[kMaxDevices] = {};      // the attribute is a per-device setting
  int dev = 0;
  cudaError_t e0 = cudaGetDevice(&dev);
  if (e0 != cudaSuccess) return e0;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!configured[dev]) {
    cudaError_t e = allow_smem(scan_gram_kernel<64, false>, kSmemBytes);
    if (e == cudaSuccess) e = allow_smem(scan_gram_kernel<32, false>, kSmemBytes);
    if (e == cudaSuccess) e = allow_smem(scan_gram_kernel<64, true>, kSmemBytes);
    if (e == cudaSuccess) e = allow_smem(scan_gram_kernel<32, true>, kSmemBytes);
    if (e == cudaSuccess) e = allow_smem(scan_gram_compact_kernel<false>, GL<true>::kBytes);
    if (e == cudaSuccess) e = allow_smem(scan_gram_compact_kernel<true>, GL<true>::kBytes);
    if (e == cudaSuccess) e = allow_smem(scan_gram_kernel<64, true, true>, kSmemBytes);
    if (e == cudaSuccess) e = allow_smem(scan_gram_kernel<32, true, true>, kSmemBytes);
    if (e == cudaSuccess) e = allow_smem(scan_gram_compact_kernel<true, true>, GL<true>::kBytes);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  // two CTAs per SM by construction: 102 KB of shared memory, 128 registers x 256 threads and 256
  // of the 512 tensor-memory columns each
  // Compact CTAs (68 KB, 80 registers, 128 tensor-memory columns: three per SM) pay one more tensor-core
  // round trip per item: they win when a launch has several waves of items (the 48-layer stack: 205 ->
  // 190 us) and lose on a single wave (batch 1: 9.3 -> 10.5 us).
  if (t.max_group_nodes <= 32 && items >= 4 * sm_count) {
    auto k = tail == 2 ? scan_gram_compact_kernel<true, true> : direct ? scan_gram_compact_kernel<true> : scan_gram_compact_kernel<false>;
    return launch_kernel(k, dim3(3 * sm_count), dim3(kThreads), GL<true>::kBytes, st, pdl, s, t, lb, items);
  }
  const int grid = items < 2 * sm_count ? items : 2 * sm_count;
  auto k = t.max_group_nodes <= 32 ? (direct ? scan_gram_kernel<32, true> : scan_gram_kernel<32, false>)
                                   : (direct ? scan_gram_kernel<64, true> : scan_gram_kernel<64, false>);
  if (tail == 2) k = t.max_group_nodes <= 32 ? scan_gram_kernel<32, true, true> : scan_gram_kernel<64, true, true>;
  return launch_kernel(k, dim3(grid), dim3(kThreads), kSmemBytes, st, pdl, s, t, lb, items);
}

cudaError_t launch_scan_gram_fused(const Shape& s, const TreeDev& t, const LayerBatch& lb, const FusedPrev& fp,
                                   int sm_count, bool pdl, int tail, cudaStream_t st) {
  const bool direct = tail != 0;
  const int items = s.n_layers * t.n_groups * s.Hv;
  static bool configured[kMaxDevices] = {};      // the attribute is a per-device setting
  int dev = 0;
  cudaError_t e0 = cudaGetDevice(&dev);
  if (e0 != cudaSuccess) return e0;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!configured[dev]) {
    cudaError_t e = allow_smem(scan_gram_fused_kernel<64, false>, kSmemBytesFused);
    if (e == cudaSuccess) e = allow_smem(scan_gram_fused_kernel<32, false>, kSmemBytesFused);
    if (e == cudaSuccess) e = allow_smem(scan_gram_fused_kernel<64, true>, kSmemBytesFused);
    if (e == cudaSuccess) e = allow_smem(scan_gram_fused_kernel<32, true>, kSmemBytesFused);
    if (e == cudaSuccess) e = allow_smem(scan_gram_fused_kernel<64, true, true>, kSmemBytesFused);
    if (e == cudaSuccess) e = allow_smem(scan_gram_fused_kernel<32, true, true>, kSmemBytesFused);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  const int grid = items < 2 * sm_count ? items : 2 * sm_count;
  auto k = t.max_group_nodes <= 32 ? (direct ? scan_gram_fused_kernel<32, true> : scan_gram_fused_kernel<32, false>)
                                   : (direct ? scan_gram_fused_kernel<64, true> : scan_gram_fused_kernel<64, false>);
  if (tail == 2) k = t.max_group_nodes <= 32 ? scan_gram_fused_kernel<32, true, true> : scan_gram_fused_kernel<64, true, true>;
  return launch_kernel(k, dim3(grid), dim3(kThreads), kSmemBytesFused, st, pdl, s, t, lb, items, fp);
}

}  // namespace lumo
