// Tree scan in solved Gram form on the 5th-generation tensor cores (tcgen05 + TMEM), sm_100a.
//
// Exact algebra of the recurrence (paper Eq. 2-3), no approximation.  With k^, q^ the scaled
// key/query of a node, G(t,s) the product of alpha over the nodes after s up to t on the path to t,
// g_t = G from the pre-tree state S0, and r_s = beta_s v_s - (beta_s g_s) S0 k^_s:
//
//   delta_t = r_t - sum_{s strict ancestor of t} A[t,s] delta_s,   A[t,s] = beta_t G(t,s) (k^_s . k^_t)
//   o_t     = g_t S0 q^_t + sum_{s ancestor of t or t itself} W[t,s] delta_s,   W[t,s] = G(t,s) (k^_s . q^_t)
//
// (the ancestor-masked triangular system the paper cites as prior art for tree verification).  The
// system couples NODES only, not value rows, so it is solved once per (sequence, value head) on scalars:
// T = (I + A)^-1 and M = W T are ancestor-masked [nodes x depth] tables, built level by level from the
// Gram products.  What is left touches d^2 data only through dense products, all on tcgen05.mma with
// fp32 accumulators in tensor memory:
//
//   Gram  = [K ; Q] K^T                                         exact products of bf16 inputs
//   q~_t  = (g_t |q scale|) q_t - sum_s M[t,s] (beta_s g_s |k scale|) k_s     "effective query", fp32 FMAs
//   O^T   = S0 q~^T  +  V^T (M diag(beta))^T                    [128 value rows x 64 nodes]
//
// S0 and q~ enter as exact bf16 hi + lo pairs (three products, the lo x lo one dropped), M diag(beta) as
// three bf16 terms (V is O(1), so its factor is carried to fp32 accuracy).  No step after the state has
// arrived is sequential over the tree: one product, one read-out, one store.  The only sequential part,
// the level loop over the scalar tables, runs while the state is still in flight.
//
// One CTA (256 threads) handles one (layer, node group, value head) at a time, two CTAs per SM.  The
// state crosses shared memory one 64-column half at a time (the second half is converted while the
// tensor core works on the first), which keeps a CTA at 110 KB.  Limits: d = 128, bf16 operands, groups
// of at most 64 nodes (larger trees are cut into groups on the host), depth <= 16, no snapshots.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "internal.h"

namespace lumo {

namespace {

constexpr int kD = 128;
constexpr int kNT = 64;               // node tile
constexpr int kThreads = 256;
constexpr int kTmemCols = 128;        // O^T: columns 0..63, Gram: columns 64..127
constexpr uint32_t kSpinLimit = 1u << 24;
constexpr uint32_t kSpinLimitDrill = 1u << 10;

// shared memory map (bytes from a 1024-aligned base)
//   region P, first life: scalar tables of the solve; second life: one 64-column half of S0 as bf16 hi + lo
constexpr int kOffP = 0;
constexpr int kOffA = kOffP;                          // [64][16] A along each node's ancestry
constexpr int kOffW = kOffP + 4096;                   // [64][16] W along each node's ancestry
constexpr int kOffCk = kOffP + 8192;                  // [64][16] -M[t,s] beta_s g_s |k scale|
constexpr int kOffDumpQ = kOffP + 12288;              // [64 columns][64 rows] Q.K products out of tensor memory
constexpr int kOffPrev = kOffP;                       // fused mode, before the tables: the previous cycle's accepted path
constexpr int kOffS0hi = kOffP, kOffS0lo = kOffP + 16384;
static_assert(kOffDumpQ + 64 * 64 * 4 <= 32768, "Q.K staging overflows region P");
//   region KQ: rows 0..63 = K, 64..127 = Q, 2 k-blocks x [128 rows x 128 B], SW128; later q~ hi + lo,
//   each 2 k-blocks x [64 rows x 128 B]
constexpr int kOffKQ = 32768;
constexpr int kOffQthi = kOffKQ, kOffQtlo = kOffKQ + 16384;
constexpr int kOffV = 65536;                          // V rows, 2 halves of 64 value columns x [64 rows x 128 B], SW128
//   region Mb, first life: [64 columns][64 rows] K.K products out of tensor memory; second life:
//   M diag(beta) as 3 bf16 terms x [64 rows x 128 B], SW128
constexpr int kOffMb = 81920;
constexpr int kOffDumpK = kOffMb;
constexpr int kOffSmall = 106496;

struct Small {
  float alpha[kNT], beta[kNT], qq[kNT], cq[kNT], ck[kNT];
  int32_t meta[kNT];                 // physical row | depth << 16 | emit << 24
  uint32_t out_off[kNT];             // element offset of the node's output row (value row 0); ~0 = not written here
  uint8_t anc[kNT][16];              // positions of the ancestors, root first, then the node itself; 0 beyond
  int32_t prev_phys[kFusedMaxPath];  // fused mode: physical rows of the previous cycle's accepted nodes
  unsigned long long mbar;
  uint32_t tmem_base;
  uint32_t timed_out;
};
constexpr int kSmemBytes = kOffSmall + (int)sizeof(Small) + 1024;   // + alignment slack
static_assert(kSmemBytes <= 113 * 1024, "two CTAs must share an SM");

// fused commit + verify: the previous cycle's accepted path and its operands for this (sequence, head)
struct PrevStage {
  int32_t acc[kFusedMaxPath], par[kFusedMaxPath], phys[kFusedMaxPath];
  float ks[kFusedMaxPath];           // key normalisation factor of each accepted node
  float2 gates[kFusedMaxPath];       // alpha, beta
  __align__(16) __nv_bfloat16 k[kFusedMaxPath][kD];
  __align__(16) __nv_bfloat16 v[kFusedMaxPath][kD];
};
static_assert(kOffPrev + (int)sizeof(PrevStage) <= kOffKQ, "path staging overflows region P");

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(gmem) : "memory");
}
// pull of the 128-byte line at `gmem` into L2 (a request without a destination register)
__device__ __forceinline__ void prefetch_l2(const void* gmem) {
  asm volatile("prefetch.global.L2 [%0];\n" ::"l"(gmem) : "memory");
}
__device__ __forceinline__ void st_zero16(uint32_t dst) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};\n" ::"r"(dst), "r"(0u) : "memory");
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(count) : "memory");
  asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
}
// Bounded wait: returns false if the phase did not complete within the spin limit.
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity, uint32_t limit) {
  const uint32_t addr = smem_u32(bar);
  for (uint32_t spin = 0; spin < limit; ++spin) {
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

// Shared-memory operand descriptor, 128-byte swizzle, version 1 (sm_100).  K-major operands: rows of
// 128 B, 8-row groups `sbo` bytes apart, `lbo` unused.  MN-major operands (the contraction index runs
// over the rows): 64 elements of the M/N dimension per 128-byte row, 8-row groups of the contraction
// index `sbo` bytes apart, the next 64 elements of the M/N dimension `lbo` bytes on.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);          // start address
  d |= (uint64_t)(lbo >> 4) << 16;                  // leading byte offset
  d |= (uint64_t)(sbo >> 4) << 32;                  // stride byte offset
  d |= (uint64_t)1 << 46;                           // descriptor version
  d |= (uint64_t)2 << 61;                           // SWIZZLE_128B
  return d;
}
__device__ __forceinline__ uint64_t desc_k(uint32_t saddr) { return umma_desc(saddr, 16, 1024); }
// kind::f16, bf16 x bf16 -> fp32; a_mn = 1: the A operand is MN-major
__host__ __device__ constexpr uint32_t umma_idesc(int M, int N, int a_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
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

__device__ __forceinline__ uint32_t sw128_offset(int row, int chunk16) {   // within one [rows x 128 B] block
  return (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((chunk16 ^ (row & 7)) << 4));
}

__device__ __forceinline__ void store_out_scalar(void* out, size_t idx, int dtype, float v) {
  if (dtype == LUMO_BF16) reinterpret_cast<__nv_bfloat16*>(out)[idx] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(out)[idx] = v;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// fp32 x -> bf16 hi + lo of four values: 8 bytes each into the hi tile and the lo tile (+16 KB)
__device__ __forceinline__ void split_store4(unsigned char* hi_tile, uint32_t off, float4 x) {
  const uint32_t h01 = pack_bf16(x.x, x.y), h23 = pack_bf16(x.z, x.w);
  const uint32_t l01 = pack_bf16(x.x - bf16_lo(h01), x.y - bf16_hi(h01));
  const uint32_t l23 = pack_bf16(x.z - bf16_lo(h23), x.w - bf16_hi(h23));
  *reinterpret_cast<uint2*>(hi_tile + off) = make_uint2(h01, h23);
  *reinterpret_cast<uint2*>(hi_tile + 16384 + off) = make_uint2(l01, l23);
}

// Element (row r, column c) of a [64 x 64] block of Gram products staged column by column: a warp
// stores one column of 32 rows without bank conflicts, and the readers (one row, the columns of its
// ancestors) spread over the banks as well.
__device__ __forceinline__ int gram_idx(int r, int c) { return c * 64 + (r ^ (c & 31)); }

// kFused: before anything else the previous cycle's accepted path is replayed into the state rows (same
// per-token update as the commit kernel) and the rows are written back in place; the scan then runs
// from the updated state.  One group per sequence only.
// kEarly: the first half of the state is requested ahead of the dependency wait (launches that overlap
// their predecessor); otherwise the key and query rows, which the longest chain of the item hangs on,
// are requested first.
template <bool kFused>
__device__ __forceinline__ void scan_solve_body(const Shape& s, const TreeDev& t, const LayerBatch& lb, int n_items,
                                                int s0_early, const FusedPrev* fp) {
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment for the swizzled operand tiles; plain pointer arithmetic on the shared
  // array keeps the pointers in the shared address space
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  Small& sm = *reinterpret_cast<Small*>(smem + kOffSmall);
  float* Am = reinterpret_cast<float*>(smem + kOffA);        // [64][16]
  float* Wm = reinterpret_cast<float*>(smem + kOffW);        // [64][16]
  float* Ck = reinterpret_cast<float*>(smem + kOffCk);       // [64][16]
  float* dumpK = reinterpret_cast<float*>(smem + kOffDumpK); // [64][64], gram_idx
  float* dumpQ = reinterpret_cast<float*>(smem + kOffDumpQ); // [64][64], gram_idx

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int grp = tid >> 7;            // half of the CTA: 0 or 1
  const int vrow = tid & 127;          // value row = TMEM lane
  const int rep = s.Hv / s.Hk;
  const bool drill = s.debug_skip_mma != 0;      // test aid: no tensor-core work is issued, the wait runs out
  const uint32_t spin_limit = drill ? kSpinLimitDrill : kSpinLimit;
  const bool early = !kFused && s0_early != 0;
  const bool one_group = t.n_groups == s.B;      // every sequence is one group: group index = sequence

  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&sm.tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  if (tid == 0) { mbar_init(&sm.mbar, 1); sm.timed_out = 0; }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  const uint32_t tmem_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16);   // this warp's 32 lanes
  uint32_t phase = 0;

  // state rows of this thread: r = 16 u + 2 warp + (lane >> 4), four floats at column 4 (lane & 15) of
  // each 64-column half
  const int srow0 = 2 * warp + (lane >> 4), c4 = lane & 15;
  const uint32_t s0_off0 = sw128_offset(srow0, c4 >> 1) + (c4 & 1) * 8;   // rows 16 u on: + 2048 u

  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {   // bounded: n_items
    const int hv = item % s.Hv;
    const int gi = (item / s.Hv) % t.n_groups;                     // node group
    const int layer = item / (s.Hv * t.n_groups);
    // the group's tables need only its index: requested before anything that has to be waited for
    int meta_r = 0;
    uint4 anc_r = make_uint4(0, 0, 0, 0);
    if (tid < kNT) meta_r = t.tc_meta[gi * kNT + tid];
    else if (tid < 2 * kNT) anc_r = *reinterpret_cast<const uint4*>(t.tc_anc + ((size_t)gi * kNT + tid - kNT) * 16);
    int b = gi, N = s.N;
    bool first_group = true;                                       // writes the per-sequence zero rows
    if (!one_group) {
      const int4 ginfo = *reinterpret_cast<const int4*>(t.tc_group + gi * 4);
      b = ginfo.x; N = ginfo.y; first_group = ginfo.z != 0;       // sequence, nodes in this group
    }
    const LayerPtrs& L = lb.l[layer];
    const int g = hv / rep;
    const int row = L.state_row[b];
    const size_t out_row_stride = (size_t)s.Hv * kD;
    // The item this CTA takes next: its state and its key, query and value rows are pulled into L2 while
    // this item computes (requests issued in phase b), so that its own loads find them there.  Only
    // lanes that issue a request look the addresses up.
    const int nxt = item + (int)gridDim.x;
    const bool has_next = !kFused && nxt < n_items;
    int n_hv = 0, n_layer = 0, n_b = 0, n_meta = -1, n_row = -1;
    if (has_next) {
      n_hv = nxt % s.Hv;
      const int n_gi = (nxt / s.Hv) % t.n_groups;
      n_layer = nxt / (s.Hv * t.n_groups);
      n_b = n_gi;
      int n_N = s.N;
      if (!one_group) { const int4 gi4 = *reinterpret_cast<const int4*>(t.tc_group + n_gi * 4); n_b = gi4.x; n_N = gi4.y; }
      if (tid < n_N) n_meta = t.tc_meta[n_gi * kNT + tid];
      n_row = lb.l[n_layer].state_row[n_b];
    }

    if (row < 0 || row >= s.n_state_rows) {   // skipped sequence: zero outputs
      pdl_wait();                             // every path through the kernel passes its dependency wait
      if (first_group) {
        for (int ps = grp; ps < s.Ns; ps += 2)
          store_out_scalar(L.out, ((size_t)b * s.Ns + ps) * out_row_stride + hv * kD + vrow, s.out_dtype, 0.f);
        if (L.status && hv == 0 && tid == 0) L.status[b] = row < 0 ? LUMO_SEQ_OK : LUMO_SEQ_BAD_ROW;
        if constexpr (kFused) {
          int32_t* pst = fp->lb.l[layer].status;
          if (pst && hv == 0 && tid == 0) pst[b] = row < 0 ? LUMO_SEQ_OK : LUMO_SEQ_BAD_ROW;
        }
      }
      continue;
    }
    if (first_group && L.status && hv == 0 && tid == 0) L.status[b] = LUMO_SEQ_OK;

    const int nmma = ((N + 15) >> 4) << 4;                         // node extent of the tensor-core products
    const float* S0 = L.state + ((size_t)row * s.Hv + hv) * kD * kD;
    float4 x0[8], x1[8];
    // The pre-tree state is not written by the kernel before this one and its address needs no table:
    // a launch that overlaps its predecessor requests the first 64-column half at once, ahead of the
    // dependency wait (two rows of 256 bytes per warp instruction).
    if (early) {
#pragma unroll
      for (int u = 0; u < 8; ++u) x0[u] = *reinterpret_cast<const float4*>(S0 + (size_t)(16 * u + srow0) * kD + 4 * c4);
    }

    int plen = 0;
    bool replay = false;
    if constexpr (kFused) {
      // ---- fused prologue: the previous cycle's commit.  The accepted path (entries, parents, physical
      // rows: one level of dependent loads) is validated by every CTA exactly as the commit kernel does;
      // the recorded key and value rows of the accepted nodes are staged, the state rows take the updates
      // u_r = S_r . k, delta_r = beta (v_r - alpha ks u_r), S_r <- alpha S_r + delta_r ks k in registers and
      // go back to memory; the scan below reads them again from there.
      pdl_wait();      // a fused launch rewrites the state: everything before it has to be complete
      PrevStage& ps = *reinterpret_cast<PrevStage*>(smem + kOffPrev);
      const LayerPtrs& PL = fp->lb.l[layer];
      plen = fp->len[b];
      const int lcap = plen < 0 ? 0 : (plen > fp->lmax ? 0 : plen);
      if (tid < lcap) {
        const int a = fp->accepted[(size_t)b * fp->lmax + tid];
        const bool ok = a >= 0 && a < fp->N;
        ps.acc[tid] = a;
        ps.par[tid] = ok ? fp->parent[(size_t)b * fp->N + a] : -2;
        const int ph = ok ? fp->slot[(size_t)b * fp->N + a] : 0;
        ps.phys[tid] = ph;
        sm.prev_phys[tid] = ph;
      }
      __syncthreads();
      const int st = check_path_staged(ps.acc, ps.par, fp->N, plen, fp->lmax);    // same answer in every thread
      if (PL.status && hv == 0 && tid == 0) PL.status[b] = st;
      replay = st == LUMO_SEQ_OK && plen > 0;
      if (replay) {
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
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          x0[u] = *reinterpret_cast<const float4*>(S0 + (size_t)(16 * u + srow0) * kD + 4 * c4);
          x1[u] = *reinterpret_cast<const float4*>(S0 + (size_t)(16 * u + srow0) * kD + 64 + 4 * c4);
        }
      }
      __syncthreads();
      if (replay) {
        for (int tt = warp; tt < plen; tt += kThreads / 32) {        // bounded: <= 16
          const uint2 w = *reinterpret_cast<const uint2*>(&ps.k[tt][4 * lane]);
          const float k0 = bf16_lo(w.x), k1 = bf16_hi(w.x), k2 = bf16_lo(w.y), k3 = bf16_hi(w.y);
          float kk = fmaf(k0, k0, fmaf(k1, k1, fmaf(k2, k2, k3 * k3)));
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) kk += __shfl_xor_sync(0xffffffffu, kk, o);
          if (lane == 0) ps.ks[tt] = s.l2norm ? rsqrtf(kk + s.l2_eps) : 1.f;
        }
      }
      __syncthreads();
      if (replay) {
        // rows r = 16 u + srow0; a row's 128 values sit in the 16 lanes of one half-warp (x0: columns
        // 4 c4 .., x1: columns 64 + 4 c4 ..)
        for (int tt = 0; tt < plen; ++tt) {                          // bounded: <= 16
          const uint2 w0 = *reinterpret_cast<const uint2*>(&ps.k[tt][4 * c4]);
          const uint2 w1 = *reinterpret_cast<const uint2*>(&ps.k[tt][64 + 4 * c4]);
          const float4 ka = make_float4(bf16_lo(w0.x), bf16_hi(w0.x), bf16_lo(w0.y), bf16_hi(w0.y));
          const float4 kb4 = make_float4(bf16_lo(w1.x), bf16_hi(w1.x), bf16_lo(w1.y), bf16_hi(w1.y));
          const float a = ps.gates[tt].x, bt = ps.gates[tt].y, ksn = ps.ks[tt];
          float p[8];
#pragma unroll
          for (int u = 0; u < 8; ++u)
            p[u] = fmaf(x0[u].x, ka.x, fmaf(x0[u].y, ka.y, fmaf(x0[u].z, ka.z, fmaf(x0[u].w, ka.w,
                   fmaf(x1[u].x, kb4.x, fmaf(x1[u].y, kb4.y, fmaf(x1[u].z, kb4.z, x1[u].w * kb4.w)))))));
#pragma unroll
          for (int o = 8; o > 0; o >>= 1)
#pragma unroll
            for (int u = 0; u < 8; ++u) p[u] += __shfl_xor_sync(0xffffffffu, p[u], o);
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const float vv = __bfloat162float(ps.v[tt][16 * u + srow0]);
            const float gk = bt * (vv - a * (ksn * p[u])) * ksn;
            x0[u].x = fmaf(a, x0[u].x, gk * ka.x); x0[u].y = fmaf(a, x0[u].y, gk * ka.y);
            x0[u].z = fmaf(a, x0[u].z, gk * ka.z); x0[u].w = fmaf(a, x0[u].w, gk * ka.w);
            x1[u].x = fmaf(a, x1[u].x, gk * kb4.x); x1[u].y = fmaf(a, x1[u].y, gk * kb4.y);
            x1[u].z = fmaf(a, x1[u].z, gk * kb4.z); x1[u].w = fmaf(a, x1[u].w, gk * kb4.w);
          }
        }
        // back in place; the same thread reads the same addresses again further down
        float* Sw = const_cast<float*>(S0);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          *reinterpret_cast<float4*>(Sw + (size_t)(16 * u + srow0) * kD + 4 * c4) = x0[u];
          *reinterpret_cast<float4*>(Sw + (size_t)(16 * u + srow0) * kD + 64 + 4 * c4) = x1[u];
        }
      }
      __syncthreads();      // the staged path is dead: the tables below take its place
    }

    // ---- a. per-node tables (the addresses of everything else depend on them) -------------------
    if (tid < kNT) {
      const int meta = tid < N ? meta_r : 0;
      sm.meta[tid] = meta;
      // a prefix node that another group emits is computed here but not written
      sm.out_off[tid] = (tid < N && ((meta >> 24) & 1)) ? (uint32_t)((((size_t)b * s.Ns + (meta & 0xFFFF)) * s.Hv + hv) * kD) : 0xFFFFFFFFu;
    } else if (tid < 2 * kNT) {
      const int pi = tid - kNT;
      *reinterpret_cast<uint4*>(sm.anc[pi]) = pi < N ? anc_r : make_uint4(0, 0, 0, 0);
    }
    __syncthreads();
    // ---- b. gates; K, Q and V rows -> swizzled operand tiles (cp.async) -------------------------------
    // K, Q, V may still be in the making (the convolution runs right before this kernel): everything
    // above touched only the descriptor tables and the state.  The dependent kernel (commit) is let in
    // afterwards: it reads freely and writes only behind its own wait.
    // A fused launch rewrites the state, which a dependent (a commit, the next scan) requests ahead of
    // its own wait: it lets nobody in before it has finished.
    if constexpr (!kFused) { pdl_wait(); pdl_trigger(); }
    if constexpr (kFused) {
      // The convolution before this kernel read the committed history through the path; now that it has
      // finished, the history buffer itself is brought up to date: the value heads of a sequence share
      // out the channels, a thread moves its 16 bytes of all three rows (reads before writes).
      if (fp->hist_in_kernels && replay && warp == kThreads / 32 - 1) {
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
            const __nv_bfloat16* src = q < 3 ? hist + (size_t)q * s.C : xprev + (size_t)sm.prev_phys[q - 3] * s.C;
            rows3[j] = *reinterpret_cast<const uint4*>(src + c * 8);
          }
#pragma unroll
          for (int j = 0; j < 3; ++j) *reinterpret_cast<uint4*>(hist + (size_t)j * s.C + c * 8) = rows3[j];
        }
      }
    }
    {
      const __nv_bfloat16* kg = reinterpret_cast<const __nv_bfloat16*>(L.k);
      const __nv_bfloat16* qg = reinterpret_cast<const __nv_bfloat16*>(L.q);
      const __nv_bfloat16* vg = reinterpret_cast<const __nv_bfloat16*>(L.v);
      // 16-byte pieces of the K and Q rows (8 per thread), then of the V rows (4 per thread): two groups,
      // so that the Gram product can start when K and Q have landed.  Copy i of a thread takes piece
      // c = tid & 15 of node (tid >> 4) + 16 (i & 3): K for i < 4, Q for i < 8, then V.
      const int c = tid & 15, nb = tid >> 4;
      const uint32_t dkq = sbase + kOffKQ + (c >> 3) * 16384, dv = sbase + kOffV + (c >> 3) * 8192;
      const size_t kq_col = (size_t)g * kD + c * 8, v_col = (size_t)hv * kD + c * 8;
      size_t pr[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) pr[i] = (size_t)b * s.Ns + (sm.meta[nb + 16 * i] & 0xFFFF);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int pi = nb + 16 * (i & 3);
        const uint32_t dst = dkq + sw128_offset(pi + (i < 4 ? 0 : kNT), c & 7);
        if (pi < N) cp_async16(dst, (i < 4 ? kg : qg) + pr[i & 3] * s.Hk * kD + kq_col);
        else if (pi < nmma) st_zero16(dst);                          // rows the products read must be finite
      }
      asm volatile("cp.async.commit_group;\n" ::: "memory");
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int pi = nb + 16 * i;
        const uint32_t dst = dv + sw128_offset(pi, c & 7);
        if (pi < N) cp_async16(dst, vg + pr[i] * s.Hv * kD + v_col);
        else if (pi < nmma) st_zero16(dst);
      }
      asm volatile("cp.async.commit_group;\n" ::: "memory");
    }
    if (!early) {
#pragma unroll
      for (int u = 0; u < 8; ++u) x0[u] = *reinterpret_cast<const float4*>(S0 + (size_t)(16 * u + srow0) * kD + 4 * c4);
    }
    if (has_next) {
      if (n_meta >= 0) {      // a node's key, query and value rows: 256 bytes = two lines each
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
    if (tid < kNT) {
      float2 gates = make_float2(1.f, 0.f);
      if (tid < N) gates = load_gates(L, s, ((size_t)b * s.Ns + (sm.meta[tid] & 0xFFFF)) * s.Hv + hv, hv);
      sm.alpha[tid] = gates.x;
      sm.beta[tid] = gates.y;
    }
    // padding rows: zero outputs
    if (first_group && s.Ns > s.N)
      for (int ps = grp; ps < s.Ns; ps += 2)
        if (t.slot_inv[b * s.Ns + ps] < 0)
          store_out_scalar(L.out, ((size_t)b * s.Ns + ps) * out_row_stride + hv * kD + vrow, s.out_dtype, 0.f);
    asm volatile("cp.async.wait_group 1;\n" ::: "memory");     // K and Q have landed (V may still be on its way)
    fence_async_proxy();          // generic-proxy writes -> visible to the tensor core's async proxy
    __syncthreads();
    // ---- c. Gram = [K;Q] K^T on the tensor core; meanwhile |q|^2 when normalising --------------------
    if (tid == 0) {
      if (!drill) {
        tc_fence_after();
        const uint32_t idesc_g = umma_idesc(128, nmma, 0);
        const uint64_t d_kq = desc_k(sbase + kOffKQ);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t koff = (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
          umma(tmem + 64, d_kq + koff, d_kq + koff, idesc_g, ks ? 1u : 0u);
        }
        umma_commit(&sm.mbar);
      }
    } else if (grp == 1 && s.l2norm && vrow < kNT) {
      const int R = kNT + vrow;   // tile row of q_vrow (the tensor core only reads the tile)
      float qq = 0.f;
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const uint4 w = *reinterpret_cast<const uint4*>(smem + kOffKQ + (c >> 3) * 16384 + sw128_offset(R, c & 7));
        const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          qq = fmaf(bf16_lo(ws[e]), bf16_lo(ws[e]), qq);
          qq = fmaf(bf16_hi(ws[e]), bf16_hi(ws[e]), qq);
        }
      }
      sm.qq[vrow] = qq;
    }
    if (warp == 0 && !mbar_wait(&sm.mbar, phase, spin_limit)) sm.timed_out = 1;   // one warp polls, the rest wait below
    phase ^= 1;
    tc_fence_after();
    __syncthreads();
    if (sm.timed_out) {    // give up on this and all further items; report, free TMEM, leave
      if (L.status && tid == 0) L.status[b] = LUMO_SEQ_TIMEOUT;
      break;
    }
    // ---- d. the Gram products leave tensor memory: lane r < 64 holds K_r . K_*, lane 64 + r holds
    //         Q_r . K_*; each half of the CTA takes 32 columns --------------------------------------------
    if (grp * 32 < N) {
      uint32_t r0[16], r1[16];
      tmem_ld16_issue(tmem_lane + 64 + grp * 32, r0);
      tmem_ld16_issue(tmem_lane + 64 + grp * 32 + 16, r1);
      tmem_ld_wait();
      float* dst = vrow < kNT ? dumpK : dumpQ;
      const int r = vrow & (kNT - 1);
#pragma unroll
      for (int e = 0; e < 16; ++e) dst[gram_idx(r, grp * 32 + e)] = __uint_as_float(r0[e]);
#pragma unroll
      for (int e = 0; e < 16; ++e) dst[gram_idx(r, grp * 32 + 16 + e)] = __uint_as_float(r1[e]);
    }
    __syncthreads();
    // ---- f. A and W along each node's ancestry, sixteen lanes per node (lane j = ancestor j, root first,
    //         the node itself last): G(t, a_j) is a suffix product of the alphas over the lanes -----------
    {
      const int j = tid & 15, ln = tid >> 4;
#pragma unroll
      for (int m = 0; m < 4; ++m) {
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
        if (s.l2norm && in) ksa = rsqrtf(dumpK[gram_idx(a, a)] + s.l2_eps);
        const float ks_t = __shfl_sync(0xffffffffu, ksa, D > 0 ? D - 1 : 0, 16);
        const float qs_t = s.l2norm ? s.scale * rsqrtf(sm.qq[pi] + s.l2_eps) : s.scale;
        const float b_t = sm.beta[pi];
        float kk = 0.f, qk = 0.f;
        if (in) { kk = dumpK[gram_idx(pi, a)]; qk = dumpQ[gram_idx(pi, a)]; }
        Am[pi * 16 + j] = j < D - 1 ? b_t * excl * ks_t * ksa * kk : 0.f;   // no entry for the node itself
        Wm[pi * 16 + j] = in ? qs_t * excl * ksa * qk : 0.f;
        if (j == 0) { sm.cq[pi] = g_t * qs_t; sm.ck[pi] = b_t * g_t * ks_t; }
      }
    }
    __syncthreads();
    // ---- g. M = W (I + A)^-1 by back substitution, independently per node (four lanes hold its 16 entries):
    //         m[j] = W[t][j] - sum_{i > j} m[i] A[anc_i][j], from the node itself up to the root.  Row anc_i of
    //         A is zero from entry i on, so every step is a plain 16-wide update.  Meanwhile the tiles of
    //         M diag(beta) are cleared (the K.K products they held are dead) -------------------------------
    for (int i = tid; i < 3 * nmma * 8; i += kThreads) {             // bounded: <= 6 rounds; rows below nmma of the three tiles
      const int term = i / (nmma * 8);
      st_zero16(sbase + kOffMb + term * 8192 + (i - term * nmma * 8) * 16);
    }
    float4 w;
    {
      const int pi = tid >> 2, q4 = tid & 3;
      const int D = pi < N ? ((sm.meta[pi] >> 16) & 0xFF) : 0;
      w = *reinterpret_cast<const float4*>(Wm + pi * 16 + 4 * q4);
      const int Dw = __reduce_max_sync(0xffffffffu, D);
      for (int jh = Dw - 1; jh >= 1; --jh) {                         // bounded: <= 15 steps
        const int e = jh & 3;
        const float cand = e == 0 ? w.x : e == 1 ? w.y : e == 2 ? w.z : w.w;
        const float mval = __shfl_sync(0xffffffffu, cand, (lane & ~3) | (jh >> 2));
        if (jh < D) {
          const float4 ar = *reinterpret_cast<const float4*>(Am + sm.anc[pi][jh] * 16 + 4 * q4);
          w.x = fmaf(-mval, ar.x, w.x); w.y = fmaf(-mval, ar.y, w.y);
          w.z = fmaf(-mval, ar.z, w.z); w.w = fmaf(-mval, ar.w, w.w);
        }
      }
    }
    __syncthreads();
    // ---- h. the two coefficient tables M feeds: Ck[t][j] = -M[t][j] beta_s g_s |k scale| (the key rows in the
    //         effective query) and M[t][j] beta_s as three bf16 terms in the operand tiles [node t][node s]
    //         of the V product ------------------------------------------------------------------------------
    {
      const int pi = tid >> 2, q4 = tid & 3;
      const int D = pi < N ? ((sm.meta[pi] >> 16) & 0xFF) : 0;
      const uint32_t a4 = *reinterpret_cast<const uint32_t*>(&sm.anc[pi][4 * q4]);
      const float mv[4] = {w.x, w.y, w.z, w.w};
      float cv[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int sidx = (a4 >> (8 * e)) & 0xFF;
        cv[e] = -mv[e] * sm.ck[sidx];                                // entries beyond the depth: M = 0
        if (4 * q4 + e < D) {
          const float mb = mv[e] * sm.beta[sidx];
          const __nv_bfloat16 h0 = __float2bfloat16_rn(mb);
          const float r1 = mb - __bfloat162float(h0);
          const __nv_bfloat16 h1 = __float2bfloat16_rn(r1);
          const __nv_bfloat16 h2 = __float2bfloat16_rn(r1 - __bfloat162float(h1));
          unsigned char* el = smem + kOffMb + sw128_offset(pi, sidx >> 3) + (sidx & 7) * 2;
          *reinterpret_cast<__nv_bfloat16*>(el) = h0;
          *reinterpret_cast<__nv_bfloat16*>(el + 8192) = h1;
          *reinterpret_cast<__nv_bfloat16*>(el + 16384) = h2;
        }
      }
      *reinterpret_cast<float4*>(Ck + pi * 16 + 4 * q4) = make_float4(cv[0], cv[1], cv[2], cv[3]);
    }
    __syncthreads();
    // ---- i. effective queries q~_t = cq_t q_t + sum_j Ck[t][j] k_{anc_j}: a thread owns 8 columns of four
    //         nodes and keeps the results in registers until every thread has finished reading K and Q ----
    float qt[4][8];
    {
      const int c = tid & 15, tb = tid >> 4;
      const uint32_t kb = kOffKQ + (c >> 3) * 16384;
      const int c7 = c & 7;
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        if (16 * m >= N) break;                                      // uniform: node rows beyond nmma are never read
        const int pi = tb + 16 * m;
        const int D = pi < N ? ((sm.meta[pi] >> 16) & 0xFF) : 0;
        float2 acc[4];
        {
          const int R = kNT + pi;
          const uint4 wq = *reinterpret_cast<const uint4*>(smem + kb + sw128_offset(R, c7));
          const float cqv = pi < N ? sm.cq[pi] : 0.f;
          acc[0] = make_float2(cqv * bf16_lo(wq.x), cqv * bf16_hi(wq.x));
          acc[1] = make_float2(cqv * bf16_lo(wq.y), cqv * bf16_hi(wq.y));
          acc[2] = make_float2(cqv * bf16_lo(wq.z), cqv * bf16_hi(wq.z));
          acc[3] = make_float2(cqv * bf16_lo(wq.w), cqv * bf16_hi(wq.w));
        }
        for (int jb = 0; jb < D; jb += 4) {                          // bounded: <= 4 blocks of four ancestors
          const uint32_t a4 = *reinterpret_cast<const uint32_t*>(&sm.anc[pi][jb]);
          const float4 c4v = *reinterpret_cast<const float4*>(Ck + pi * 16 + jb);
          const float cf[4] = {c4v.x, c4v.y, c4v.z, c4v.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {                              // entries beyond the depth: coefficient 0, row 0
            const int a = (a4 >> (8 * e)) & 0xFF;
            const uint4 wk = *reinterpret_cast<const uint4*>(smem + kb + (a << 7) + ((c7 ^ (a & 7)) << 4));
            const float2 cc = make_float2(cf[e], cf[e]);
            acc[0] = __ffma2_rn(cc, make_float2(bf16_lo(wk.x), bf16_hi(wk.x)), acc[0]);
            acc[1] = __ffma2_rn(cc, make_float2(bf16_lo(wk.y), bf16_hi(wk.y)), acc[1]);
            acc[2] = __ffma2_rn(cc, make_float2(bf16_lo(wk.z), bf16_hi(wk.z)), acc[2]);
            acc[3] = __ffma2_rn(cc, make_float2(bf16_lo(wk.w), bf16_hi(wk.w)), acc[3]);
          }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) { qt[m][2 * e] = acc[e].x; qt[m][2 * e + 1] = acc[e].y; }
      }
    }
    __syncthreads();      // K, Q and the scalar tables are dead from here on
    // second 64-column half of the state: in flight while the first is converted and multiplied
#pragma unroll
    for (int u = 0; u < 8; ++u) x1[u] = *reinterpret_cast<const float4*>(S0 + (size_t)(16 * u + srow0) * kD + 64 + 4 * c4);
    // ---- j. q~ -> bf16 hi + lo operand tiles [node][128 columns] in the place of K and Q ----------------
    {
      const int c = tid & 15, tb = tid >> 4;
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        if (16 * m >= N) break;                                      // uniform
        const int pi = tb + 16 * m;
        uint32_t h[4], l[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          h[e] = pack_bf16(qt[m][2 * e], qt[m][2 * e + 1]);
          l[e] = pack_bf16(qt[m][2 * e] - bf16_lo(h[e]), qt[m][2 * e + 1] - bf16_hi(h[e]));
        }
        const uint32_t off = (c >> 3) * 8192 + sw128_offset(pi, c & 7);
        *reinterpret_cast<uint4*>(smem + kOffQthi + off) = make_uint4(h[0], h[1], h[2], h[3]);
        *reinterpret_cast<uint4*>(smem + kOffQtlo + off) = make_uint4(l[0], l[1], l[2], l[3]);
      }
    }
    // ---- l. first half of the state -> bf16 hi + lo tiles; products of that half and the V product -------
#pragma unroll
    for (int u = 0; u < 8; ++u) split_store4(smem + kOffS0hi, s0_off0 + 2048 * u, x0[u]);
    asm volatile("cp.async.wait_group 0;\n" ::: "memory");     // the V rows have landed
    fence_async_proxy();
    __syncthreads();
    const int nks_v = (N + 15) >> 4;                                 // 16-node steps of the V product
    if (tid == 0 && !drill) {
      tc_fence_after();
      const uint32_t idesc_o = umma_idesc(128, nmma, 0), idesc_v = umma_idesc(128, nmma, 1);
      const uint64_t d_hi = desc_k(sbase + kOffS0hi), d_lo = desc_k(sbase + kOffS0lo);
      const uint64_t d_qh = desc_k(sbase + kOffQthi), d_ql = desc_k(sbase + kOffQtlo);
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        const uint64_t koff = (uint64_t)((ks * 32) >> 4);
        umma(tmem, d_hi + koff, d_qh + koff, idesc_o, ks ? 1u : 0u);
        umma(tmem, d_hi + koff, d_ql + koff, idesc_o, 1u);
        umma(tmem, d_lo + koff, d_qh + koff, idesc_o, 1u);
      }
      // V^T (MN-major A: 64 value columns per 128-byte row, 8-node groups 1024 B apart, the other 64
      // columns 8192 B on) times the three terms of M diag(beta) (K-major B)
      for (int ks = 0; ks < nks_v; ++ks) {                           // bounded: <= 4
        const uint64_t d_v = umma_desc(sbase + kOffV + ks * 2048, 8192, 1024);
#pragma unroll
        for (int r = 0; r < 3; ++r) umma(tmem, d_v, desc_k(sbase + kOffMb + r * 8192 + ks * 32), idesc_v, 1u);
      }
      umma_commit(&sm.mbar);
    }
    if (warp == 0 && !mbar_wait(&sm.mbar, phase, spin_limit)) sm.timed_out = 1;   // one warp polls, the rest wait below
    phase ^= 1;
    tc_fence_after();
    __syncthreads();
    if (sm.timed_out) {
      if (L.status && tid == 0) L.status[b] = LUMO_SEQ_TIMEOUT;
      break;
    }
    // ---- m. second half of the state through the same tiles ----------------------------------------------
#pragma unroll
    for (int u = 0; u < 8; ++u) split_store4(smem + kOffS0hi, s0_off0 + 2048 * u, x1[u]);
    fence_async_proxy();
    __syncthreads();
    if (tid == 0 && !drill) {
      tc_fence_after();
      const uint32_t idesc_o = umma_idesc(128, nmma, 0);
      const uint64_t d_hi = desc_k(sbase + kOffS0hi), d_lo = desc_k(sbase + kOffS0lo);
      const uint64_t d_qh = desc_k(sbase + kOffQthi + 8192), d_ql = desc_k(sbase + kOffQtlo + 8192);
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        const uint64_t koff = (uint64_t)((ks * 32) >> 4);
        umma(tmem, d_hi + koff, d_qh + koff, idesc_o, 1u);
        umma(tmem, d_hi + koff, d_ql + koff, idesc_o, 1u);
        umma(tmem, d_lo + koff, d_qh + koff, idesc_o, 1u);
      }
      umma_commit(&sm.mbar);
    }
    if (warp == 0 && !mbar_wait(&sm.mbar, phase, spin_limit)) sm.timed_out = 1;   // one warp polls, the rest wait below
    phase ^= 1;
    tc_fence_after();
    __syncthreads();
    if (sm.timed_out) {
      if (L.status && tid == 0) L.status[b] = LUMO_SEQ_TIMEOUT;
      break;
    }
    // ---- n. outputs: lane = value row, column = node; each half of the CTA takes 32 nodes ---------------
    if (grp * 32 < N) {
      uint32_t r0[16], r1[16];
      tmem_ld16_issue(tmem_lane + grp * 32, r0);
      tmem_ld16_issue(tmem_lane + grp * 32 + 16, r1);
      tmem_ld_wait();
      if (s.out_dtype == LUMO_BF16) {
        __nv_bfloat16* outp = reinterpret_cast<__nv_bfloat16*>(L.out) + vrow;
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const uint32_t oo = sm.out_off[grp * 32 + e];
          if (oo != 0xFFFFFFFFu) outp[oo] = __float2bfloat16_rn(__uint_as_float(r0[e]));
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const uint32_t oo = sm.out_off[grp * 32 + 16 + e];
          if (oo != 0xFFFFFFFFu) outp[oo] = __float2bfloat16_rn(__uint_as_float(r1[e]));
        }
      } else {
        float* outp = reinterpret_cast<float*>(L.out) + vrow;
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const uint32_t oo = sm.out_off[grp * 32 + e];
          if (oo != 0xFFFFFFFFu) outp[oo] = __uint_as_float(r0[e]);
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const uint32_t oo = sm.out_off[grp * 32 + 16 + e];
          if (oo != 0xFFFFFFFFu) outp[oo] = __uint_as_float(r1[e]);
        }
      }
    }
    tc_fence_before();
    __syncthreads();      // tensor memory and the shared memory are free for the next item
  }

  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

__global__ void __launch_bounds__(kThreads, 2)
scan_solve_kernel(Shape s, TreeDev t, LayerBatch lb, int n_items, int s0_early) {
  scan_solve_body<false>(s, t, lb, n_items, s0_early, nullptr);
}

__global__ void __launch_bounds__(kThreads, 2)
scan_solve_fused_kernel(Shape s, TreeDev t, LayerBatch lb, int n_items, FusedPrev fp) {
  scan_solve_body<true>(s, t, lb, n_items, 0, &fp);
}

template <typename K>
cudaError_t configure_once(K kern, bool (&done)[kMaxDevices]) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!done[dev]) {                          // the attribute is a per-device setting
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    done[dev] = true;
  }
  return cudaSuccess;
}

}  // namespace

cudaError_t launch_scan_solve(const Shape& s, const TreeDev& t, const LayerBatch& lb, int sm_count, bool pdl,
                              cudaStream_t st) {
  const int items = s.n_layers * t.n_groups * s.Hv;
  static bool configured[kMaxDevices] = {};
  cudaError_t e = configure_once(scan_solve_kernel, configured);
  if (e != cudaSuccess) return e;
  // two CTAs per SM by construction: 110 KB of shared memory, 128 registers x 256 threads and 128
  // of the 512 tensor-memory columns each
  const int grid = items < 2 * sm_count ? items : 2 * sm_count;
  return launch_kernel(scan_solve_kernel, dim3(grid), dim3(kThreads), kSmemBytes, st, pdl, s, t, lb, items, pdl ? 1 : 0);
}

cudaError_t launch_scan_solve_fused(const Shape& s, const TreeDev& t, const LayerBatch& lb, const FusedPrev& fp,
                                    int sm_count, bool pdl, cudaStream_t st) {
  const int items = s.n_layers * t.n_groups * s.Hv;
  static bool configured[kMaxDevices] = {};
  cudaError_t e = configure_once(scan_solve_fused_kernel, configured);
  if (e != cudaSuccess) return e;
  const int grid = items < 2 * sm_count ? items : 2 * sm_count;
  return launch_kernel(scan_solve_fused_kernel, dim3(grid), dim3(kThreads), kSmemBytes, st, pdl, s, t, lb, items, fp);
}

}  // namespace lumo
