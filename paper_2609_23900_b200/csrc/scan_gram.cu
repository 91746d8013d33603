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
// Everything after that is O(depth) fp32 FMAs per (row, node): thread r owns value row r (= TMEM
// lane r), keeps the deltas of the current root-to-node path in registers indexed by depth, and
// walks the nodes in depth-first order, so sequential fp32 arithmetic along each path is kept.
//
// One CTA (128 threads) handles one (layer, sequence, value head) at a time; two CTAs per SM
// overlap one item's loads with the other's arithmetic.  Limits of this kernel: d = 128, bf16
// operands, N <= 64 nodes, tree depth <= 16, no state snapshots; everything else takes the
// rank-1 kernel.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "internal.h"

namespace lumo {

namespace {

constexpr int kD = 128;
constexpr int kNT = 64;               // node tile
constexpr int kThreads = 128;
constexpr int kTmemCols = 256;        // P: 128 columns, Gram: 64 columns (power of two allocation)
constexpr int kWStride = 20;          // floats per coefficient row: 16 W, c0, beta/unused, depth bits, pad
constexpr int kDumpStride = 68;       // floats per dumped Gram row (conflict-free 128-bit stores)
constexpr uint32_t kSpinLimit = 1u << 24;

// shared memory map (bytes from a 1024-aligned base)
constexpr int kOffAhi = 0;                          // S0 hi: 2 k-blocks x [128 rows x 128 B], SW128
constexpr int kOffAlo = 32768;                      // S0 lo
constexpr int kOffKQ = 65536;                       // rows 0..63 = K, 64..127 = Q, 2 k-blocks, SW128
constexpr int kOffSmall = 98304;
// after the MMAs have completed the S0 tiles are dead; their space is reused:
constexpr int kOffDump = 0;                         // Gram [128][68] fp32
constexpr int kOffWk = kOffDump + 128 * kDumpStride * 4;   // 34816
constexpr int kOffWq = kOffWk + kNT * kWStride * 4;        // 39936
constexpr int kOffV = kOffWq + kNT * kWStride * 4;         // 45056: V [64][128] bf16
static_assert(kOffV + kNT * kD * 2 <= kOffKQ, "aliased region overflows the S0 tiles");

struct Small {
  float alpha[kNT], beta[kNT], ks[kNT], qs[kNT];
  int32_t meta[kNT];                 // physical row | depth << 16
  uint8_t anc[kNT][16];              // depth-first positions of the ancestors, root first
  unsigned long long mbar;
  uint32_t tmem_base;
  uint32_t timed_out;
};
constexpr int kSmemBytes = kOffSmall + (int)sizeof(Small) + 1024;   // + alignment slack

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit_wait_all() {
  asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
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
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ uint32_t sw128_offset(int row, int chunk16) {   // within one [rows x 128 B] k-block
  return (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((chunk16 ^ (row & 7)) << 4));
}

__device__ __forceinline__ void store_out(void* out, size_t idx, int dtype, float v) {
  if (dtype == LUMO_BF16) reinterpret_cast<__nv_bfloat16*>(out)[idx] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(out)[idx] = v;
}

template <int DMAX>
__global__ void __launch_bounds__(kThreads, 2)
scan_gram_kernel(Shape s, TreeDev t, LayerBatch lb, int n_items) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  Small& sm = *reinterpret_cast<Small*>(smem + kOffSmall);
  float* dump = reinterpret_cast<float*>(smem + kOffDump);
  float* Wk = reinterpret_cast<float*>(smem + kOffWk);
  float* Wq = reinterpret_cast<float*>(smem + kOffWq);
  const __nv_bfloat16* Vs = reinterpret_cast<const __nv_bfloat16*>(smem + kOffV);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rep = s.Hv / s.Hk;
  const int N = s.N;

  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&sm.tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  if (tid == 0) { mbar_init(&sm.mbar, 1); sm.timed_out = 0; }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  const uint32_t tmem_lane = tmem + ((uint32_t)(warp * 32) << 16);   // this warp's 32 lanes
  uint32_t phase = 0;

  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {   // bounded: n_items
    const int hv = item % s.Hv;
    const int b = (item / s.Hv) % s.B;
    const int layer = item / (s.Hv * s.B);
    const LayerPtrs& L = lb.l[layer];
    const int g = hv / rep;
    const int row = L.state_row[b];
    const size_t out_row_stride = (size_t)s.Hv * kD;

    if (row < 0 || row >= s.n_state_rows) {   // skipped sequence: zero outputs
      for (int ps = 0; ps < s.Ns; ++ps) store_out(L.out, ((size_t)b * s.Ns + ps) * out_row_stride + hv * kD + tid, s.out_dtype, 0.f);
      if (L.status && hv == 0 && tid == 0) L.status[b] = row < 0 ? LUMO_SEQ_OK : LUMO_SEQ_BAD_ROW;
      continue;
    }
    if (L.status && hv == 0 && tid == 0) L.status[b] = LUMO_SEQ_OK;

    // ---- a. per-node tables and gates -----------------------------------------------------
    if (tid < kNT) {
      const int pi = tid;
      int meta = 0;
      float a = 1.f, bt = 0.f;
      if (pi < N) {
        meta = t.tc_meta[b * N + pi];
        const size_t pr = (size_t)b * s.Ns + (meta & 0xFFFF);
        a = s.gate_dtype == LUMO_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(L.alpha)[pr * s.Hv + hv])
                                      : reinterpret_cast<const float*>(L.alpha)[pr * s.Hv + hv];
        bt = s.gate_dtype == LUMO_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(L.beta)[pr * s.Hv + hv])
                                       : reinterpret_cast<const float*>(L.beta)[pr * s.Hv + hv];
      }
      sm.meta[pi] = meta; sm.alpha[pi] = a; sm.beta[pi] = bt;
    } else {
      const int pi = tid - kNT;
      uint4 av = make_uint4(0, 0, 0, 0);
      if (pi < N) av = *reinterpret_cast<const uint4*>(t.tc_anc + ((size_t)b * N + pi) * 16);
      *reinterpret_cast<uint4*>(sm.anc[pi]) = av;
    }
    // padding rows: zero outputs
    if (s.Ns > N)
      for (int ps = 0; ps < s.Ns; ++ps)
        if (t.slot_inv[b * s.Ns + ps] < 0)
        store_out(L.out, ((size_t)b * s.Ns + ps) * out_row_stride + hv * kD + tid, s.out_dtype, 0.f);
    __syncthreads();

    // ---- b. K and Q rows -> swizzled operand tile (cp.async) -------------------------------
    {
      const __nv_bfloat16* kg = reinterpret_cast<const __nv_bfloat16*>(L.k);
      const __nv_bfloat16* qg = reinterpret_cast<const __nv_bfloat16*>(L.q);
#pragma unroll 4
      for (int i = 0; i < 16; ++i) {
        const int idx = i * kThreads + tid;
        const int R = idx >> 4, c = idx & 15;
        const int pi = R & (kNT - 1);
        const uint32_t dst = sbase + kOffKQ + (c >> 3) * 16384 + sw128_offset(R, c & 7);
        if (pi < N) {
          const size_t pr = (size_t)b * s.Ns + (sm.meta[pi] & 0xFFFF);
          const __nv_bfloat16* src = (R < kNT ? kg : qg) + (pr * s.Hk + g) * kD + c * 8;
          cp_async16(dst, src);
        } else {
          asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};\n" ::"r"(dst), "r"(0u) : "memory");
        }
      }
    }
    // ---- c. S0 -> bf16 hi + lo operand tiles ------------------------------------------------
    {
      const float* S0 = L.state + ((size_t)row * s.Hv + hv) * kD * kD;
      const int kblock = lane >> 4, chunk = (lane & 15) >> 1, half = lane & 1;
#pragma unroll 1
      for (int i0 = 0; i0 < 32; i0 += 8) {
        float4 x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = *reinterpret_cast<const float4*>(S0 + (size_t)(warp * 32 + i0 + u) * kD + lane * 4);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int r = warp * 32 + i0 + u;
          __nv_bfloat162 h01 = __floats2bfloat162_rn(x[u].x, x[u].y), h23 = __floats2bfloat162_rn(x[u].z, x[u].w);
          float2 f01 = __bfloat1622float2(h01), f23 = __bfloat1622float2(h23);
          __nv_bfloat162 l01 = __floats2bfloat162_rn(x[u].x - f01.x, x[u].y - f01.y);
          __nv_bfloat162 l23 = __floats2bfloat162_rn(x[u].z - f23.x, x[u].w - f23.y);
          const uint32_t off = kblock * 16384 + sw128_offset(r, chunk) + half * 8;
          *reinterpret_cast<uint2*>(smem + kOffAhi + off) =
              make_uint2(*reinterpret_cast<uint32_t*>(&h01), *reinterpret_cast<uint32_t*>(&h23));
          *reinterpret_cast<uint2*>(smem + kOffAlo + off) =
              make_uint2(*reinterpret_cast<uint32_t*>(&l01), *reinterpret_cast<uint32_t*>(&l23));
        }
      }
    }
    cp_async_commit_wait_all();
    fence_async_proxy();          // generic-proxy writes -> visible to the tensor core's async proxy
    __syncthreads();

    // ---- e. MMAs: P = S0 [K|Q]^T (hi + lo), Gram = [K;Q] K^T --------------------------------
    if (tid == 0) {
      tc_fence_after();
      constexpr uint32_t idesc_p = umma_idesc(128, 128), idesc_g = umma_idesc(128, 64);
#pragma unroll
      for (int term = 0; term < 2; ++term) {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint32_t koff = (ks >> 2) * 16384 + (ks & 3) * 32;
          umma(tmem, umma_desc(sbase + (term ? kOffAlo : kOffAhi) + koff), umma_desc(sbase + kOffKQ + koff), idesc_p,
               (term | ks) ? 1u : 0u);
        }
      }
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const uint32_t koff = (ks >> 2) * 16384 + (ks & 3) * 32;
        umma(tmem + 128, umma_desc(sbase + kOffKQ + koff), umma_desc(sbase + kOffKQ + koff), idesc_g, ks ? 1u : 0u);
      }
      umma_commit(&sm.mbar);
    }
    // ---- f. wait for the tensor core (bounded) ----------------------------------------------
    if (!mbar_wait(&sm.mbar, phase)) sm.timed_out = 1;
    phase ^= 1;
    tc_fence_after();
    __syncthreads();
    if (sm.timed_out) {    // give up on this and all further items; report, free TMEM, leave
      if (L.status && tid == 0) L.status[b] = LUMO_SEQ_TIMEOUT;
      break;
    }

    // ---- g. V rows -> shared (space of the dead S0 tiles) ----------------------------------
    {
      const __nv_bfloat16* vg = reinterpret_cast<const __nv_bfloat16*>(L.v);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int idx = i * kThreads + tid;
        const int pi = idx >> 4, c = idx & 15;
        if (pi < N) {
          const size_t pr = (size_t)b * s.Ns + (sm.meta[pi] & 0xFFFF);
          cp_async16(sbase + kOffV + pi * 256 + c * 16, vg + (pr * s.Hv + hv) * kD + c * 8);
        }
      }
      asm volatile("cp.async.commit_group;\n" ::: "memory");
    }
    // ---- h. Gram rows out of tensor memory; |q|^2 when normalising ----------------------------
    {
      float gr[16];
#pragma unroll
      for (int cb = 0; cb < 4; ++cb) {
        tmem_ld16(tmem_lane + 128 + cb * 16, gr);
#pragma unroll
        for (int e = 0; e < 16; e += 4)
          *reinterpret_cast<float4*>(dump + tid * kDumpStride + cb * 16 + e) = make_float4(gr[e], gr[e + 1], gr[e + 2], gr[e + 3]);
      }
    }
    float qq = 0.f;
    if (s.l2norm && tid >= kNT) {
      const int R = tid;   // tile row of q_(tid-64)
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const uint4 w = *reinterpret_cast<const uint4*>(smem + kOffKQ + (c >> 3) * 16384 + sw128_offset(R, c & 7));
        const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float lo = __uint_as_float(ws[e] << 16), hi = __uint_as_float(ws[e] & 0xFFFF0000u);
          qq = fmaf(lo, lo, qq); qq = fmaf(hi, hi, qq);
        }
      }
    }
    __syncthreads();
    // ---- i. normalisation factors ----------------------------------------------------------
    if (tid < kNT) sm.ks[tid] = s.l2norm ? rsqrtf(dump[tid * kDumpStride + tid] + s.l2_eps) : 1.f;
    else sm.qs[tid - kNT] = s.l2norm ? s.scale * rsqrtf(qq + s.l2_eps) : s.scale;
    __syncthreads();
    // ---- j. coefficient rows: one thread per (node, table) ------------------------------------
    {
      const bool is_q = tid >= kNT;
      const int pi = tid & (kNT - 1);
      float w[kWStride];
#pragma unroll
      for (int e = 0; e < kWStride; ++e) w[e] = 0.f;
      if (pi < N) {
        const int D = sm.meta[pi] >> 16;                         // depth, 1..16
        const float a_t = sm.alpha[pi], b_t = sm.beta[pi];
        const float self = is_q ? sm.qs[pi] : b_t * sm.ks[pi];   // factor of the node itself
        const float* grow = dump + (is_q ? kNT + pi : pi) * kDumpStride;
        float G = a_t;
#pragma unroll
        for (int j = 15; j >= 0; --j) {                          // bounded: 16 depth slots
          if (j <= D - 2) {
            const int sidx = sm.anc[pi][j];
            w[j] = self * G * sm.ks[sidx] * grow[sidx];
            G *= sm.alpha[sidx];
          }
        }
        if (is_q) {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (j == D - 1) w[j] = self * sm.ks[pi] * grow[pi];   // k^_t . q^_t, G = 1
        }
        w[16] = self * G;                                         // factor of the S0 product
        w[17] = b_t;
        w[18] = __int_as_float(D);
      }
      float* dst = (is_q ? Wq : Wk) + pi * kWStride;
#pragma unroll
      for (int e = 0; e < kWStride; e += 4) *reinterpret_cast<float4*>(dst + e) = make_float4(w[e], w[e + 1], w[e + 2], w[e + 3]);
    }
    asm volatile("cp.async.wait_group 0;\n" ::: "memory");
    __syncthreads();

    // ---- k. forward substitution along the depth-first walk: thread = value row --------------
    {
      float dl[DMAX];
#pragma unroll
      for (int j = 0; j < DMAX; ++j) dl[j] = 0.f;
      const int nblk = (N + 15) >> 4;
      for (int blk = 0; blk < nblk; ++blk) {                      // bounded: <= 4
        float pk[16], pq[16];
        tmem_ld16(tmem_lane + blk * 16, pk);
        tmem_ld16(tmem_lane + kNT + blk * 16, pq);
#pragma unroll
        for (int u = 0; u < 16; ++u) {
          const int pi = blk * 16 + u;
          if (pi < N) {
            const float* wk = Wk + pi * kWStride;
            const float* wq = Wq + pi * kWStride;
            const float4 tail = *reinterpret_cast<const float4*>(wk + 16);     // c0, beta, depth
            const int D = __float_as_int(tail.z);
            const float v = __bfloat162float(Vs[pi * kD + tid]);
            float acc0 = fmaf(tail.y, v, -tail.x * pk[u]), acc1 = 0.f;
#pragma unroll
            for (int j4 = 0; j4 < DMAX; j4 += 4) {
              const float4 c = *reinterpret_cast<const float4*>(wk + j4);
              acc0 = fmaf(-c.x, dl[j4], acc0); acc1 = fmaf(-c.y, dl[j4 + 1], acc1);
              acc0 = fmaf(-c.z, dl[j4 + 2], acc0); acc1 = fmaf(-c.w, dl[j4 + 3], acc1);
            }
            const float delta = acc0 + acc1;
#pragma unroll
            for (int j = 0; j < DMAX; ++j) dl[j] = (j == D - 1) ? delta : dl[j];
            float o0 = wq[16] * pq[u], o1 = 0.f;
#pragma unroll
            for (int j4 = 0; j4 < DMAX; j4 += 4) {
              const float4 c = *reinterpret_cast<const float4*>(wq + j4);
              o0 = fmaf(c.x, dl[j4], o0); o1 = fmaf(c.y, dl[j4 + 1], o1);
              o0 = fmaf(c.z, dl[j4 + 2], o0); o1 = fmaf(c.w, dl[j4 + 3], o1);
            }
            const size_t pr = (size_t)b * s.Ns + (sm.meta[pi] & 0xFFFF);
            store_out(L.out, pr * out_row_stride + hv * kD + tid, s.out_dtype, o0 + o1);
          }
        }
      }
    }
    tc_fence_before();
    __syncthreads();      // tensor memory and the aliased shared memory are free for the next item
  }

  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

}  // namespace

bool gram_supported(const Shape& s, int max_depth) {
  return s.d == kD && s.in_dtype == LUMO_BF16 && s.snapshot_mode == 0 && s.N <= kNT && max_depth <= 16;
}

cudaError_t launch_scan_gram(const Shape& s, const TreeDev& t, const LayerBatch& lb, int max_depth, int sm_count,
                             cudaStream_t st) {
  const int items = s.n_layers * s.B * s.Hv;
  const int grid = items < 2 * sm_count ? items : 2 * sm_count;
  auto launch = [&](auto kern) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    kern<<<grid, kThreads, kSmemBytes, st>>>(s, t, lb, items);
    return cudaGetLastError();
  };
  if (max_depth <= 4) return launch(scan_gram_kernel<4>);
  if (max_depth <= 8) return launch(scan_gram_kernel<8>);
  return launch(scan_gram_kernel<16>);
}

}  // namespace lumo
