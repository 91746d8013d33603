// sm_100a kernels of the GDN tree verifier: tree convolution, rank-1 tree scan, commit.
//
// Row independence is what the layout is built on: row r of the d_v x d_k state evolves
// alone (S[r,:] <- a S[r,:] + delta_r k^T with delta_r = b (v_r - a S[r,:].k)), so a CTA
// owns 32 rows of one (sequence, value head) and walks the WHOLE tree with them, four lanes
// per row, each lane holding d_k/4 fp32 state values in registers (paper Eq. 2-3; Sec.
// "Path-parallel verification and state lifetime": the working tile keeps the full key
// dimension and is reused along the path instead of being reloaded per node).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <climits>
#include <mutex>
#include <type_traits>

#include "internal.h"

namespace lumo {

namespace {

constexpr int kRows = 32;        // state rows per CTA
constexpr int kLanesPerRow = 4;
constexpr int kScanThreads = kRows * kLanesPerRow;   // 128
constexpr int kRingDepth = 6;    // staged node operands in flight

// ---------------------------------------------------------------------------------------
// small helpers
// ---------------------------------------------------------------------------------------
template <typename T> struct Vec4;   // four consecutive elements -> float4
template <> struct Vec4<float> {
  static __device__ __forceinline__ float4 load(const float* p) { return *reinterpret_cast<const float4*>(p); }
};
template <> struct Vec4<__nv_bfloat16> {
  static __device__ __forceinline__ float4 load(const __nv_bfloat16* p) {
    uint2 r = *reinterpret_cast<const uint2*>(p);
    return make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xFFFF0000u),
                       __uint_as_float(r.y << 16), __uint_as_float(r.y & 0xFFFF0000u));
  }
};

__device__ __forceinline__ void store_scalar(void* p, size_t i, int dtype, float v) {
  if (dtype == LUMO_BF16) reinterpret_cast<__nv_bfloat16*>(p)[i] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(p)[i] = v;
}

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  unsigned s = (unsigned)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

__device__ __forceinline__ float ex2_approx(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float rcp_approx(float x) { float y; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

template <typename T> struct Packed4;      // four consecutive elements as loaded
template <> struct Packed4<float> {
  using type = float4;
  static __device__ __forceinline__ float4 unpack(const float4& p) { return p; }
};
template <> struct Packed4<__nv_bfloat16> {
  using type = uint2;
  static __device__ __forceinline__ float4 unpack(const uint2& r) {
    return make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xFFFF0000u),
                       __uint_as_float(r.y << 16), __uint_as_float(r.y & 0xFFFF0000u));
  }
};

// ---------------------------------------------------------------------------------------
// a1: ancestry-gathered causal depthwise conv (width 4) + SiLU -> recorded operands
// ---------------------------------------------------------------------------------------
// A CTA owns kConvRows consecutive entries of one sequence's visiting order (depth-first, built on
// the host) and a slab of 256 x 4 channels; a thread keeps the taps (as pairs of neighbouring
// channels), the bias and the current 4-row window of its channels unpacked in fp32 registers.  In
// depth-first order most rows either follow their parent (the window slides by one) or share the
// parent of the previous row (only the own row changes), so one load per row replaces four; the own
// rows of the next eight entries are always in flight (the kernel is bound by the special-function
// unit, two operations per element for the SiLU, and by load latency, not by bandwidth).  Windows
// that cannot be derived come from a table in the same visiting order (physical rows, or -1..-3 for
// the history rows), fetched together with the order itself.
// Taps are applied oldest first in fp32 starting from zero (packed FMAs: two correctly rounded fp32
// lanes per instruction, same bits as scalar fmaf), bias last, SiLU in fp32, one round-to-nearest-even
// cast (Sec. "Precompute branch histories while preserving arithmetic": tap order and cast points are
// part of the result).

// kFused: the three history rows are the ones the previous cycle's accepted path will commit, i.e. the
// last three of [old history ; raw inputs of the accepted nodes], read in place through the path (the
// scan that follows writes them to the history buffer once every CTA of this kernel has finished).
template <typename T, int kConvRows, bool kFused>
__device__ __forceinline__ void conv_body(const Shape& s, const TreeDev& t, const LayerBatch& lb, const FusedPrev* fp) {
  __shared__ int s_win[kConvRows][4];
  __shared__ int s_prog[kConvRows];
  __shared__ int f_acc[kFusedMaxPath], f_par[kFusedMaxPath], f_phys[kFusedMaxPath];
  __shared__ const T* f_hsrc[3];
  const int layer = blockIdx.z / s.B, b = blockIdx.z % s.B;
  const int e0 = blockIdx.y * kConvRows;               // first entry of the visiting order
  const int c0 = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  const LayerPtrs& L = lb.l[layer];
  pdl_wait();       // x, history and the operand buffers belong to earlier kernels until here
  pdl_trigger();
  const int row = L.state_row[b];
  const bool seq_ok = row >= 0 && row < s.n_state_rows;
  if (threadIdx.x < kConvRows * 4) {
    const int r = threadIdx.x >> 2, j = threadIdx.x & 3;
    int prog = 3 << 16, w = INT_MIN;
    if (e0 + r < s.Ns) {
      prog = t.conv_prog[(size_t)b * s.Ns + e0 + r];
      if (!seq_ok) prog = (prog & 0xFFFF) | (3 << 16);        // skipped sequence: every row is a zero row
      w = t.win[((size_t)b * s.Ns + e0 + r) * 4 + j];
    }
    s_win[r][j] = w;
    if (j == 0) s_prog[r] = (e0 + r < s.Ns) ? prog : -1;
  }
  int plen = 0;
  if constexpr (kFused) {
    plen = fp->len[b];
    const int lcap = plen < 0 ? 0 : (plen > fp->lmax ? 0 : plen);
    const int tt = (int)threadIdx.x - 128;
    if (tt >= 0 && tt < lcap) {
      const int a = fp->accepted[(size_t)b * fp->lmax + tt];
      const bool ok = a >= 0 && a < fp->N;
      f_acc[tt] = a;
      f_par[tt] = ok ? fp->parent[(size_t)b * fp->N + a] : -2;
      f_phys[tt] = ok ? fp->slot[(size_t)b * fp->N + a] : 0;
    }
  }
  using P4 = typename Packed4<T>::type;                // four elements as loaded
  float2 wp[4][2];                                     // tap j of channel pairs (0,1) and (2,3)
  float2 bp[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
  if (c0 < s.C) {
    const T* w = reinterpret_cast<const T*>(L.conv_w) + (size_t)c0 * 4;
    float4 wc[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) wc[e] = Packed4<T>::unpack(*reinterpret_cast<const P4*>(w + e * 4));
    wp[0][0] = make_float2(wc[0].x, wc[1].x); wp[0][1] = make_float2(wc[2].x, wc[3].x);
    wp[1][0] = make_float2(wc[0].y, wc[1].y); wp[1][1] = make_float2(wc[2].y, wc[3].y);
    wp[2][0] = make_float2(wc[0].z, wc[1].z); wp[2][1] = make_float2(wc[2].z, wc[3].z);
    wp[3][0] = make_float2(wc[0].w, wc[1].w); wp[3][1] = make_float2(wc[2].w, wc[3].w);
    if (L.conv_b) {
      const float4 bv = Packed4<T>::unpack(*reinterpret_cast<const P4*>(reinterpret_cast<const T*>(L.conv_b) + c0));
      bp[0] = make_float2(bv.x, bv.y);
      bp[1] = make_float2(bv.z, bv.w);
    }
  }
  __syncthreads();
  if constexpr (kFused) {
    if (threadIdx.x == 0) {
      // an invalid or empty path commits nothing: the history in memory is the history
      const bool ok = seq_ok && check_path_staged(f_acc, f_par, fp->N, plen, fp->lmax) == LUMO_SEQ_OK;
      const int leff = ok ? plen : 0;
      const T* hbase = reinterpret_cast<const T*>(L.conv_hist) + (size_t)(seq_ok ? row : 0) * 3 * s.C;
      const T* xprev = reinterpret_cast<const T*>(fp->lb.l[layer].x) + (size_t)b * fp->Ns * s.C;
      for (int j = 0; j < 3; ++j) {
        const int q = leff + j;        // index into [old0 old1 old2 x_a0 x_a1 ...]
        f_hsrc[j] = q < 3 ? hbase + (size_t)q * s.C : xprev + (size_t)f_phys[q - 3] * s.C;
      }
    }
    __syncthreads();
  }
  if (c0 >= s.C) return;
  const bool has_bias = L.conv_b != nullptr;
  const int hkd = s.Hk * s.d;
  T* dst;
  size_t dst_stride;
  if (c0 < hkd) { dst = reinterpret_cast<T*>(L.q) + c0; dst_stride = hkd; }
  else if (c0 < 2 * hkd) { dst = reinterpret_cast<T*>(L.k) + (c0 - hkd); dst_stride = hkd; }
  else { dst = reinterpret_cast<T*>(L.v) + (c0 - 2 * hkd); dst_stride = (size_t)s.Hv * s.d; }
  dst += (size_t)b * s.Ns * dst_stride;
  const T* x = reinterpret_cast<const T*>(L.x) + (size_t)b * s.Ns * s.C + c0;
  const T* hist = reinterpret_cast<const T*>(L.conv_hist) + (size_t)(seq_ok ? row : 0) * 3 * s.C + c0;

  auto load_src = [&](int wj) -> float4 {              // one window entry: a row of x or of the history
    const T* src;
    if (wj >= 0) src = x + (size_t)wj * s.C;
    else if constexpr (kFused) src = f_hsrc[3 + wj] + c0;
    else src = hist + (size_t)(3 + wj) * s.C;
    return Packed4<T>::unpack(*reinterpret_cast<const P4*>(src));
  };
  auto load_own = [&](int r) -> P4 {                   // the entry's own row (padding rows: zeros)
    const int prog = r < kConvRows ? s_prog[r] : -1;
    P4 z = {};
    if (prog < 0 || (prog >> 16) == 3) return z;
    return *reinterpret_cast<const P4*>(x + (size_t)(prog & 0xFFFF) * s.C);
  };
  float4 win[4] = {};
  constexpr int kAhead = sizeof(T) == 2 ? (kConvRows < 8 ? kConvRows : 8) : 4;   // own rows in flight (a register budget)
  P4 pf[kAhead];
#pragma unroll
  for (int r = 0; r < kAhead; ++r) pf[r] = load_own(r);
#pragma unroll
  for (int r = 0; r < kConvRows; ++r) {                // bounded: kConvRows
    const int prog = s_prog[r];
    if (prog < 0) break;
    const int ps = prog & 0xFFFF;
    int flag = prog >> 16;
    if (r == 0 && flag != 3) flag = 0;                 // the first row of a CTA has nothing to reuse
    const float4 own = Packed4<T>::unpack(pf[r % kAhead]);
    pf[r % kAhead] = load_own(r + kAhead);
    float y[4] = {0.f, 0.f, 0.f, 0.f};
    if (flag != 3) {
      if (flag == 0) { win[0] = load_src(s_win[r][0]); win[1] = load_src(s_win[r][1]); win[2] = load_src(s_win[r][2]); }
      else if (flag == 1) { win[0] = win[1]; win[1] = win[2]; win[2] = win[3]; }
      win[3] = own;
      float2 y01 = make_float2(0.f, 0.f), y23 = make_float2(0.f, 0.f);
#pragma unroll
      for (int j = 0; j < 4; ++j) {                    // oldest -> newest
        y01 = __ffma2_rn(wp[j][0], make_float2(win[j].x, win[j].y), y01);
        y23 = __ffma2_rn(wp[j][1], make_float2(win[j].z, win[j].w), y23);
      }
      if (has_bias) { y01 = __fadd2_rn(y01, bp[0]); y23 = __fadd2_rn(y23, bp[1]); }   // bias last
      // SiLU a / (1 + 2^(-a log2 e)) with the hardware exponential and reciprocal (1e-6 relative, far
      // below the rounding of the recorded operand); the multiplies and the add are packed
      const float2 nl2e = make_float2(-1.4426950408889634f, -1.4426950408889634f), one = make_float2(1.f, 1.f);
      float2 e01 = __fmul2_rn(y01, nl2e), e23 = __fmul2_rn(y23, nl2e);
      e01 = __fadd2_rn(make_float2(ex2_approx(e01.x), ex2_approx(e01.y)), one);
      e23 = __fadd2_rn(make_float2(ex2_approx(e23.x), ex2_approx(e23.y)), one);
      y01 = __fmul2_rn(y01, make_float2(rcp_approx(e01.x), rcp_approx(e01.y)));
      y23 = __fmul2_rn(y23, make_float2(rcp_approx(e23.x), rcp_approx(e23.y)));
      y[0] = y01.x; y[1] = y01.y; y[2] = y23.x; y[3] = y23.y;
    }
    T* d = dst + (size_t)ps * dst_stride;
    if constexpr (sizeof(T) == 2) {
      __nv_bfloat162 h01 = __floats2bfloat162_rn(y[0], y[1]), h23 = __floats2bfloat162_rn(y[2], y[3]);
      *reinterpret_cast<uint2*>(d) = make_uint2(*reinterpret_cast<uint32_t*>(&h01), *reinterpret_cast<uint32_t*>(&h23));
    } else {
      *reinterpret_cast<float4*>(d) = make_float4(y[0], y[1], y[2], y[3]);
    }
  }
}

template <typename T, int kConvRows>
__global__ void __launch_bounds__(256, 3) conv_kernel(Shape s, TreeDev t, LayerBatch lb) {
  conv_body<T, kConvRows, false>(s, t, lb, nullptr);
}
template <typename T, int kConvRows>
__global__ void __launch_bounds__(256, 3) conv_fused_kernel(Shape s, TreeDev t, LayerBatch lb, FusedPrev fp) {
  conv_body<T, kConvRows, true>(s, t, lb, &fp);
}

// ---------------------------------------------------------------------------------------
// a3: rank-1 tree scan
// ---------------------------------------------------------------------------------------
template <int D, typename T>
struct ScanCfg {
  static constexpr int kChunks = D / 16;            // float4 chunks per lane
  static constexpr int kStageElems = 2 * D + kRows; // k row, q row, v slice
  static constexpr int kStageBytes = kStageElems * (int)sizeof(T);
  static constexpr int kStageXfers = kStageBytes / 16;
  static constexpr int kKXfers = D * (int)sizeof(T) / 16;
};

// dynamic shared memory layout (bytes), computed identically on host and device
struct ScanSmem {
  int ops, slot, params, dcache, snaplist, ring, total;
};
__host__ __device__ inline ScanSmem scan_smem(int N, int max_ops, int n_snap_list, int stage_bytes) {
  ScanSmem m;
  int off = 0;
  m.ops = off;      off += ((max_ops * 4 + 15) / 16) * 16;
  m.slot = off;     off += ((N * 4 + 15) / 16) * 16;
  m.params = off;   off += 5 * N * 4;  off = (off + 15) / 16 * 16;
  m.dcache = off;   off += N * kRows * 4;
  m.snaplist = off; off += ((n_snap_list * 4 + 15) / 16) * 16;
  m.ring = off;     off += kRingDepth * stage_bytes;
  m.total = off;
  return m;
}

template <int D, typename T>
__global__ void __launch_bounds__(kScanThreads)
scan_kernel(Shape s, TreeDev t, LayerBatch lb, float* __restrict__ stack, int n_items) {
  using Cfg = ScanCfg<D, T>;
  constexpr int NCH = Cfg::kChunks;
  extern __shared__ __align__(16) unsigned char smem[];
  const int n_snap_list = s.snapshot_mode == 1 ? s.n_snap : 0;
  const ScanSmem lay = scan_smem(s.N, t.max_ops, n_snap_list, Cfg::kStageBytes);
  int32_t* s_ops = reinterpret_cast<int32_t*>(smem + lay.ops);
  int32_t* s_slot = reinterpret_cast<int32_t*>(smem + lay.slot);   // physical row of each node
  float* p_a = reinterpret_cast<float*>(smem + lay.params);
  float* p_b = p_a + s.N;
  float* p_ks = p_b + s.N;      // multiplies the raw key (1 / norm when normalising)
  float* p_qs = p_ks + s.N;     // multiplies the raw query (scale / norm)
  float* p_kq = p_qs + s.N;     // k_n . q_n with both factors applied
  float* s_dc = reinterpret_cast<float*>(smem + lay.dcache);
  int32_t* s_snap = reinterpret_cast<int32_t*>(smem + lay.snaplist);
  unsigned char* s_ring = smem + lay.ring;

  const int tid = threadIdx.x;
  const int j = tid & 3;               // lane within the row group
  const int rl = tid >> 2;             // local row 0..31
  constexpr int kTiles = D / kRows;
  const int rep = s.Hv / s.Hk;
  float* my_stack = stack + (size_t)blockIdx.x * t.max_levels * (kRows * D);

  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {   // bounded: n_items
    const int tile = item % kTiles;
    const int hv = (item / kTiles) % s.Hv;
    const int b = (item / (kTiles * s.Hv)) % s.B;
    const int layer = item / (kTiles * s.Hv * s.B);
    const LayerPtrs& L = lb.l[layer];
    const int g = hv / rep;
    const int row = L.state_row[b];
    const int r0 = tile * kRows;
    const size_t out_row_stride = (size_t)s.Hv * D;
    __syncthreads();   // previous item's shared memory is no longer in use

    if (row < 0 || row >= s.n_state_rows) {
      // skipped sequence: zero outputs; flag a row outside the pool
      for (int e = tid; e < s.Ns * kRows; e += kScanThreads)
        store_scalar(L.out, ((size_t)b * s.Ns + e / kRows) * out_row_stride + hv * D + r0 + e % kRows,
                     s.out_dtype, 0.f);
      if (L.status && hv == 0 && tile == 0 && tid == 0) L.status[b] = row < 0 ? LUMO_SEQ_OK : LUMO_SEQ_BAD_ROW;
      continue;
    }
    if (L.status && hv == 0 && tile == 0 && tid == 0) L.status[b] = LUMO_SEQ_OK;

    // pre-tree state tile -> registers (issued first so the loads overlap the prologue)
    const float* S0 = L.state + (((size_t)row * s.Hv + hv) * D + r0 + rl) * D;
    float4 S[NCH];
#pragma unroll
    for (int m = 0; m < NCH; ++m) S[m] = *reinterpret_cast<const float4*>(S0 + 16 * m + 4 * j);

    const int nops = t.nops[b];
    const int32_t* ops_g = t.sched + (size_t)b * t.max_ops;
    for (int e = tid; e < nops; e += kScanThreads) s_ops[e] = ops_g[e];
    for (int e = tid; e < s.N; e += kScanThreads) s_slot[e] = t.slot[b * s.N + e];
    for (int e = tid; e < n_snap_list; e += kScanThreads) s_snap[e] = L.snap_nodes[(size_t)b * s.n_snap + e];
    // padding rows: zero outputs
    for (int e = tid; e < s.Ns * kRows; e += kScanThreads) {
      int ps = e / kRows;
      if (t.slot_inv[b * s.Ns + ps] < 0)
        store_scalar(L.out, ((size_t)b * s.Ns + ps) * out_row_stride + hv * D + r0 + e % kRows, s.out_dtype, 0.f);
    }
    // per-node scalars: gates, normalisation factors, k.q
    const T* qg = reinterpret_cast<const T*>(L.q);
    const T* kg = reinterpret_cast<const T*>(L.k);
    const T* vg = reinterpret_cast<const T*>(L.v);
    {
      // eight lanes per node, sixteen nodes in flight per pass; the trip count is uniform over
      // the CTA so that every lane takes part in the shuffles
      const int grp = tid >> 3, gl = tid & 7;
#pragma unroll 2
      for (int n0 = 0; n0 < s.N; n0 += kScanThreads / 8) {
        const int n = n0 + grp;
        const bool live = n < s.N;
        const size_t pr = (size_t)b * s.Ns + (live ? t.slot[b * s.N + n] : 0);
        const T* kr = kg + (pr * s.Hk + g) * D;
        const T* qr = qg + (pr * s.Hk + g) * D;
        float kk = 0.f, qq = 0.f, kq = 0.f;
        if (live) {
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            float4 kv = Vec4<T>::load(kr + gl * 4 + 32 * c), qv = Vec4<T>::load(qr + gl * 4 + 32 * c);
            kk += kv.x * kv.x + kv.y * kv.y + kv.z * kv.z + kv.w * kv.w;
            qq += qv.x * qv.x + qv.y * qv.y + qv.z * qv.z + qv.w * qv.w;
            kq += kv.x * qv.x + kv.y * qv.y + kv.z * qv.z + kv.w * qv.w;
          }
        }
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) {
          kk += __shfl_xor_sync(0xffffffffu, kk, o);
          qq += __shfl_xor_sync(0xffffffffu, qq, o);
          kq += __shfl_xor_sync(0xffffffffu, kq, o);
        }
        if (live && gl == 0) {
          float ks = 1.f, qs = s.scale;
          if (s.l2norm) { ks = rsqrtf(kk + s.l2_eps); qs = s.scale * rsqrtf(qq + s.l2_eps); }
          p_ks[n] = ks; p_qs[n] = qs; p_kq[n] = kq * ks * qs;
          const float2 gates = load_gates(L, s, pr * s.Hv + hv, hv);
          p_a[n] = gates.x;
          p_b[n] = gates.y;
        }
      }
    }
    __syncthreads();

    // operand ring: stage i holds k row, q row and this tile's v slice of op i's node
    auto prefetch = [&](int i) {
      if (i < nops) {
        const int op = s_ops[i];
        const int kind = op >> 24;
        if (kind <= OP_DESCEND) {
          const int n = op & 0xFFFF;
          const size_t pr = (size_t)b * s.Ns + s_slot[n];
          unsigned char* st = s_ring + (i % kRingDepth) * Cfg::kStageBytes;
          const int nx = kind == OP_DESCEND ? Cfg::kKXfers : Cfg::kStageXfers;
          if (tid < nx) {
            const unsigned char* src;
            if (tid < Cfg::kKXfers) src = reinterpret_cast<const unsigned char*>(kg + (pr * s.Hk + g) * D) + tid * 16;
            else if (tid < 2 * Cfg::kKXfers)
              src = reinterpret_cast<const unsigned char*>(qg + (pr * s.Hk + g) * D) + (tid - Cfg::kKXfers) * 16;
            else
              src = reinterpret_cast<const unsigned char*>(vg + (pr * s.Hv + hv) * D + r0) + (tid - 2 * Cfg::kKXfers) * 16;
            cp_async16(st + tid * 16, src);
          }
        }
      }
      cp_async_commit();
    };
#pragma unroll
    for (int i = 0; i < kRingDepth - 1; ++i) prefetch(i);

    for (int i = 0; i < nops; ++i) {                   // bounded: nops <= max_ops
      cp_async_wait<kRingDepth - 2>();
      __syncthreads();
      prefetch(i + kRingDepth - 1);
      const int op = s_ops[i];
      const int kind = op >> 24;
      const int arg = op & 0xFFFF;
      const T* st_k = reinterpret_cast<const T*>(s_ring + (i % kRingDepth) * Cfg::kStageBytes);
      const T* st_q = st_k + D;
      const T* st_v = st_q + D;
      if (kind <= OP_EMIT_DESCEND) {
        const int n = arg;
        float u0 = 0.f, u1 = 0.f, w0 = 0.f, w1 = 0.f;
#pragma unroll
        for (int m = 0; m < NCH; ++m) {
          float4 kv = Vec4<T>::load(st_k + 16 * m + 4 * j);
          float4 qv = Vec4<T>::load(st_q + 16 * m + 4 * j);
          u0 = fmaf(S[m].x, kv.x, u0); u1 = fmaf(S[m].y, kv.y, u1);
          u0 = fmaf(S[m].z, kv.z, u0); u1 = fmaf(S[m].w, kv.w, u1);
          w0 = fmaf(S[m].x, qv.x, w0); w1 = fmaf(S[m].y, qv.y, w1);
          w0 = fmaf(S[m].z, qv.z, w0); w1 = fmaf(S[m].w, qv.w, w1);
        }
        float u = u0 + u1, w = w0 + w1;
        u += __shfl_xor_sync(0xffffffffu, u, 1); w += __shfl_xor_sync(0xffffffffu, w, 1);
        u += __shfl_xor_sync(0xffffffffu, u, 2); w += __shfl_xor_sync(0xffffffffu, w, 2);
        const float a = p_a[n], bt = p_b[n], ks = p_ks[n];
        float vv;
        if constexpr (sizeof(T) == 2) vv = __bfloat162float(st_v[rl]); else vv = st_v[rl];
        const float dl = bt * (vv - a * (ks * u));          // delta = beta (v - R' k)
        const float o = a * (p_qs[n] * w) + dl * p_kq[n];   // o = R q = a R_p q + delta (k.q)
        if (j == 0) {
          const size_t pr = (size_t)b * s.Ns + s_slot[n];
          store_scalar(L.out, pr * out_row_stride + hv * D + r0 + rl, s.out_dtype, o);
          if ((op >> 20) & 1) s_dc[n * kRows + rl] = dl;
        }
        if (kind == OP_EMIT_DESCEND) {
          const float gk = dl * ks;
#pragma unroll
          for (int m = 0; m < NCH; ++m) {
            float4 kv = Vec4<T>::load(st_k + 16 * m + 4 * j);
            S[m].x = fmaf(a, S[m].x, gk * kv.x); S[m].y = fmaf(a, S[m].y, gk * kv.y);
            S[m].z = fmaf(a, S[m].z, gk * kv.z); S[m].w = fmaf(a, S[m].w, gk * kv.w);
          }
        }
      } else if (kind == OP_DESCEND) {
        const int n = arg;
        const float a = p_a[n];
        const float gk = s_dc[n * kRows + rl] * p_ks[n];
#pragma unroll
        for (int m = 0; m < NCH; ++m) {
          float4 kv = Vec4<T>::load(st_k + 16 * m + 4 * j);
          S[m].x = fmaf(a, S[m].x, gk * kv.x); S[m].y = fmaf(a, S[m].y, gk * kv.y);
          S[m].z = fmaf(a, S[m].z, gk * kv.z); S[m].w = fmaf(a, S[m].w, gk * kv.w);
        }
      } else if (kind == OP_PUSH) {
        float* dst = my_stack + ((size_t)arg * kRows + rl) * D;
#pragma unroll
        for (int m = 0; m < NCH; ++m) *reinterpret_cast<float4*>(dst + 16 * m + 4 * j) = S[m];
      } else {  // OP_POP
        const float* src = arg == kPopRoot ? S0 : my_stack + ((size_t)arg * kRows + rl) * D;
#pragma unroll
        for (int m = 0; m < NCH; ++m) S[m] = *reinterpret_cast<const float4*>(src + 16 * m + 4 * j);
      }
      // node states on request: the registers now hold S_n
      if (s.snapshot_mode != 0 && (kind == OP_EMIT_DESCEND || kind == OP_DESCEND)) {
        const int n = arg;
        const int E = s.n_snap;
        if (s.snapshot_mode == 2) {
          float* dst = L.snap_out + ((((size_t)b * E + n) * s.Hv + hv) * D + r0 + rl) * D;
#pragma unroll
          for (int m = 0; m < NCH; ++m) *reinterpret_cast<float4*>(dst + 16 * m + 4 * j) = S[m];
        } else {
          for (int e = 0; e < E; ++e) {          // bounded: E
            if (s_snap[e] != n) continue;
            float* dst = L.snap_out + ((((size_t)b * E + e) * s.Hv + hv) * D + r0 + rl) * D;
#pragma unroll
            for (int m = 0; m < NCH; ++m) *reinterpret_cast<float4*>(dst + 16 * m + 4 * j) = S[m];
          }
        }
      }
    }
    cp_async_wait<0>();
  }
}

// ---------------------------------------------------------------------------------------
// a4 + a5: commit - replay the accepted path into the running state, in place, and gather the
// convolution history of the accepted path
// ---------------------------------------------------------------------------------------
// One launch.  The first Hv * d/32 CTAs of a (sequence, layer) each own a 32-row state tile: same
// per-token arithmetic as the scan's EMIT_DESCEND without the output, i.e. the "native per-token
// update" of Algorithm 2 applied for the accepted nodes in path order.  The remaining CTAs own
// 128 x 16 bytes of channels of the history rows: new history = last three rows of
// [old history ; x of the accepted nodes] (Algorithm 1).  The state tile is requested from memory
// before the path is validated, so the two dependent chains (tile; length -> path -> operands) overlap;
// nothing is written unless the path is valid.
template <int D, typename T>
__global__ void __launch_bounds__(kScanThreads, (D == 128 && sizeof(T) == 2) ? 8 : 4)
commit_kernel(Shape s, TreeDev t, LayerBatch lb, const int32_t* __restrict__ accepted,
              const int32_t* __restrict__ len_arr, int lmax, int n_state_ctas) {
  constexpr int NCH = D / 16;
  constexpr int kTiles = D / kRows;
  using P4 = typename Packed4<T>::type;
  const int b = blockIdx.y, layer = blockIdx.z;
  const LayerPtrs& L = lb.l[layer];
  const int tid = threadIdx.x;
  const int row = L.state_row[b];
  const bool lead = blockIdx.x == 0 && tid == 0;
  // What this kernel WRITES (state, history, status) may still be read by its predecessor (the scan
  // reads the pre-tree state), so every write sits behind pdl_wait().  What it READS ahead of that wait
  // (state tile, path, operands) must be older than its predecessor: the host launches it with the
  // overlap attribute only right after a verify call, whose own dependency wait orders everything
  // before it; after any other call of the library it is launched in plain stream order.
  if (row < 0) { pdl_wait(); if (lead && L.status) L.status[b] = LUMO_SEQ_OK; return; }
  if (row >= s.n_state_rows) { pdl_wait(); if (lead && L.status) L.status[b] = LUMO_SEQ_BAD_ROW; return; }
  const int32_t* acc = accepted + (size_t)b * lmax;
  // the whole path at once: entry t, its parent and its physical row (one level of dependent loads
  // instead of one per step)
  __shared__ int s_acc[kMaxNodes], s_par[kMaxNodes], s_phys[kMaxNodes];
  const int len = len_arr[b];
  const int lcap = len < 0 ? 0 : (len > lmax ? 0 : len);
  for (int tt = tid; tt < lcap; tt += kScanThreads) {     // bounded: lmax
    const int a = acc[tt];
    const bool ok = a >= 0 && a < s.N;
    s_acc[tt] = a;
    s_par[tt] = ok ? t.parent[(size_t)b * s.N + a] : -2;
    s_phys[tt] = ok ? t.slot[b * s.N + a] : 0;
  }

  if ((int)blockIdx.x >= n_state_ctas) {
    // ---- convolution history ------------------------------------------------------------------
    constexpr int kVec = 16 / (int)sizeof(T);
    const int c0 = ((blockIdx.x - n_state_ctas) * kScanThreads + tid) * kVec;
    __syncthreads();
    // every exit path passes the dependency wait: a CTA that left without it would let this grid complete
    // (and its own dependent start) while the kernel before it is still running
    if (c0 >= s.C || L.x == nullptr) { pdl_wait(); return; }
    if (check_path_staged(s_acc, s_par, s.N, len, lmax) != LUMO_SEQ_OK || len == 0) { pdl_wait(); return; }
    T* hist = reinterpret_cast<T*>(L.conv_hist) + (size_t)row * 3 * s.C + c0;
    const T* x = reinterpret_cast<const T*>(L.x);
    uint4 v[3];
#pragma unroll
    for (int jj = 0; jj < 3; ++jj) {
      const int q = len + jj;        // index into [old0 old1 old2 x_a0 x_a1 ...]
      const T* src = q < 3 ? hist + (size_t)q * s.C
                           : x + ((size_t)b * s.Ns + s_phys[q - 3]) * s.C + c0;
      v[jj] = *reinterpret_cast<const uint4*>(src);
    }
    pdl_wait();
#pragma unroll
    for (int jj = 0; jj < 3; ++jj) *reinterpret_cast<uint4*>(hist + (size_t)jj * s.C) = v[jj];
    return;
  }

  // ---- state tile ---------------------------------------------------------------------------------
  const int tile = blockIdx.x % kTiles, hv = blockIdx.x / kTiles;
  const int j = tid & 3, rl = tid >> 2;
  const int g = hv / (s.Hv / s.Hk);
  const int r0 = tile * kRows;
  float* Sg = L.state + (((size_t)row * s.Hv + hv) * D + r0 + rl) * D;
  float4 S[NCH];
#pragma unroll
  for (int m = 0; m < NCH; ++m) S[m] = *reinterpret_cast<const float4*>(Sg + 16 * m + 4 * j);   // in flight

  __syncthreads();
  const int st = check_path_staged(s_acc, s_par, s.N, len, lmax);
  if (lead && L.status) { pdl_wait(); L.status[b] = st; }
  if (st != LUMO_SEQ_OK || len == 0) { pdl_wait(); return; }

  const T* kg = reinterpret_cast<const T*>(L.k);
  const T* vg = reinterpret_cast<const T*>(L.v);
  for (int tt = 0; tt < len; ++tt) {                      // bounded: len <= lmax
    const size_t pr = (size_t)b * s.Ns + s_phys[tt];
    const T* kr = kg + (pr * s.Hk + g) * D;
    P4 kp[NCH];
#pragma unroll
    for (int m = 0; m < NCH; ++m) kp[m] = *reinterpret_cast<const P4*>(kr + 16 * m + 4 * j);
    float vv;
    if constexpr (sizeof(T) == 2) vv = __bfloat162float(vg[(pr * s.Hv + hv) * D + r0 + rl]);
    else vv = vg[(pr * s.Hv + hv) * D + r0 + rl];
    const float2 gates = load_gates(L, s, pr * s.Hv + hv, hv);
    const float a = gates.x, bt = gates.y;
    float u0 = 0.f, u1 = 0.f, k0 = 0.f, k1 = 0.f;
#pragma unroll
    for (int m = 0; m < NCH; ++m) {
      const float4 kv = Packed4<T>::unpack(kp[m]);
      u0 = fmaf(S[m].x, kv.x, u0); u1 = fmaf(S[m].y, kv.y, u1);
      u0 = fmaf(S[m].z, kv.z, u0); u1 = fmaf(S[m].w, kv.w, u1);
      k0 = fmaf(kv.x, kv.x, k0); k1 = fmaf(kv.y, kv.y, k1);
      k0 = fmaf(kv.z, kv.z, k0); k1 = fmaf(kv.w, kv.w, k1);
    }
    float u = u0 + u1, kk = k0 + k1;
    u += __shfl_xor_sync(0xffffffffu, u, 1); kk += __shfl_xor_sync(0xffffffffu, kk, 1);
    u += __shfl_xor_sync(0xffffffffu, u, 2); kk += __shfl_xor_sync(0xffffffffu, kk, 2);
    const float ks = s.l2norm ? rsqrtf(kk + s.l2_eps) : 1.f;
    const float dl = bt * (vv - a * (ks * u));
    const float gk = dl * ks;
#pragma unroll
    for (int m = 0; m < NCH; ++m) {
      const float4 kv = Packed4<T>::unpack(kp[m]);
      S[m].x = fmaf(a, S[m].x, gk * kv.x); S[m].y = fmaf(a, S[m].y, gk * kv.y);
      S[m].z = fmaf(a, S[m].z, gk * kv.z); S[m].w = fmaf(a, S[m].w, gk * kv.w);
    }
  }
  pdl_wait();
#pragma unroll
  for (int m = 0; m < NCH; ++m) *reinterpret_cast<float4*>(Sg + 16 * m + 4 * j) = S[m];
}

// device helper: root-first path ending at node[b]
__global__ void path_from_node_kernel(TreeDev t, int B, int N, const int32_t* __restrict__ node,
                                      int lmax, int32_t* __restrict__ accepted,
                                      int32_t* __restrict__ len, int32_t* __restrict__ status) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  int32_t* acc = accepted + (size_t)b * lmax;
  for (int e = 0; e < lmax; ++e) acc[e] = -1;
  int n = node[b], st = LUMO_SEQ_OK, l = 0;
  if (n != -1) {
    if (n < 0 || n >= N) st = LUMO_SEQ_BAD_NODE;
    else {
      l = t.depth[(size_t)b * N + n];
      if (l > lmax) { st = LUMO_SEQ_BAD_LEN; l = 0; }
      else
        for (int e = l - 1; e >= 0 && n >= 0; --e) { acc[e] = n; n = t.parent[(size_t)b * N + n]; }  // bounded: depth
    }
  }
  len[b] = l;
  if (status) status[b] = st;
}

template <typename F>
cudaError_t dispatch(int d, int in_dtype, F f) {
  if (d == 128 && in_dtype == LUMO_BF16) return f(std::integral_constant<int, 128>{}, __nv_bfloat16{});
  if (d == 128 && in_dtype == LUMO_F32) return f(std::integral_constant<int, 128>{}, float{});
  if (d == 64 && in_dtype == LUMO_BF16) return f(std::integral_constant<int, 64>{}, __nv_bfloat16{});
  if (d == 64 && in_dtype == LUMO_F32) return f(std::integral_constant<int, 64>{}, float{});
  return cudaErrorInvalidValue;
}

}  // namespace

// ---------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------
// sixteen entries per CTA amortise the window set-up; small launches take fewer so that the grid still
// covers the GPU
int conv_rows_per_cta(int C, int Ns, int seqs, int sms) {
  const int slabs = (C / 4 + 255) / 256;
  auto ctas = [&](int rows) { return (long long)slabs * ((Ns + rows - 1) / rows) * seqs; };
  if (ctas(16) >= 2LL * sms) return 16;
  if (ctas(8) >= 2LL * sms) return 8;
  return 4;
}

template <typename T>
static cudaError_t launch_conv_t(const Shape& s, const TreeDev& t, const LayerBatch& lb, const FusedPrev* fp, bool pdl,
                                 cudaStream_t st) {
  const int slabs = (s.C / 4 + 255) / 256, seqs = s.B * s.n_layers;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int rows = conv_rows_per_cta(s.C, s.Ns, seqs, sms);
  auto go = [&](auto rows_c) {
    constexpr int kRowsPerCta = decltype(rows_c)::value;
    const dim3 grid(slabs, (s.Ns + kRowsPerCta - 1) / kRowsPerCta, seqs);
    if (fp) return launch_kernel(conv_fused_kernel<T, kRowsPerCta>, grid, dim3(256), 0, st, pdl, s, t, lb, *fp);
    return launch_kernel(conv_kernel<T, kRowsPerCta>, grid, dim3(256), 0, st, pdl, s, t, lb);
  };
  if (rows == 16) return go(std::integral_constant<int, 16>{});
  if (rows == 8) return go(std::integral_constant<int, 8>{});
  return go(std::integral_constant<int, 4>{});
}

cudaError_t launch_conv(const Shape& s, const TreeDev& t, const LayerBatch& lb, bool pdl, cudaStream_t st) {
  if (s.in_dtype == LUMO_BF16) return launch_conv_t<__nv_bfloat16>(s, t, lb, nullptr, pdl, st);
  return launch_conv_t<float>(s, t, lb, nullptr, pdl, st);
}

cudaError_t launch_conv_fused(const Shape& s, const TreeDev& t, const LayerBatch& lb, const FusedPrev& fp, bool pdl,
                              cudaStream_t st) {
  if (s.in_dtype != LUMO_BF16) return cudaErrorInvalidValue;      // the fused path serves bf16 operands only
  return launch_conv_t<__nv_bfloat16>(s, t, lb, &fp, pdl, st);
}

cudaError_t scan_plan(const Shape& s, const TreeDev& t, int sm_count, int* grid, size_t* stack_bytes) {
  const int items = s.n_layers * s.B * s.Hv * (s.d / kRows);
  return dispatch(s.d, s.in_dtype, [&](auto dc, auto tc) {
    constexpr int D = decltype(dc)::value;
    using T = decltype(tc);
    const int n_snap_list = s.snapshot_mode == 1 ? s.n_snap : 0;
    const ScanSmem lay = scan_smem(s.N, t.max_ops, n_snap_list, ScanCfg<D, T>::kStageBytes);
    auto kern = scan_kernel<D, T>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, lay.total);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kScanThreads, lay.total);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    const int resident = sm_count * per_sm;
    *grid = items < resident ? items : resident;
    *stack_bytes = (size_t)*grid * t.max_levels * kRows * D * sizeof(float);
    return cudaSuccess;
  });
}

// ---------------------------------------------------------------------------------------
// fixed scratch for callers that cannot allocate (lumo_gdn_tree_scan_static)
// ---------------------------------------------------------------------------------------
// The scan's state stack normally lives in memory the context allocates on first use.  This
// array is the same stack with a fixed capacity, part of the library image on every GPU that
// loads it.  Host code must not pass `g_static_stack` itself to a kernel: on the host the name
// is only a handle for the symbol, so its device address is looked up once per device.
__device__ __align__(256) static float g_static_stack[kStaticStackBytes / sizeof(float)];

cudaError_t static_stack_address(int device, float** ptr) {
  static float* cached[kMaxDevices] = {};
  static std::mutex mu;
  if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  if (!cached[device]) {
    int cur = -1;
    cudaError_t e = cudaGetDevice(&cur);
    if (e != cudaSuccess) return e;
    if (cur != device) return cudaErrorInvalidDevice;   // the caller makes `device` current first
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_stack);
    if (e != cudaSuccess) return e;
    cached[device] = static_cast<float*>(p);
  }
  *ptr = cached[device];
  return cudaSuccess;
}

cudaError_t launch_scan(const Shape& s, const TreeDev& t, const LayerBatch& lb, float* stack,
                        int grid, cudaStream_t st) {
  const int items = s.n_layers * s.B * s.Hv * (s.d / kRows);
  return dispatch(s.d, s.in_dtype, [&](auto dc, auto tc) {
    constexpr int D = decltype(dc)::value;
    using T = decltype(tc);
    const int n_snap_list = s.snapshot_mode == 1 ? s.n_snap : 0;
    const ScanSmem lay = scan_smem(s.N, t.max_ops, n_snap_list, ScanCfg<D, T>::kStageBytes);
    scan_kernel<D, T><<<grid, kScanThreads, lay.total, st>>>(s, t, lb, stack, items);
    return cudaGetLastError();
  });
}

cudaError_t launch_commit(const Shape& s, const TreeDev& t, const LayerBatch& lb, const int32_t* accepted,
                          const int32_t* len, int lmax, bool with_state, bool with_hist, bool pdl, cudaStream_t st) {
  if (!with_state && !with_hist) return cudaSuccess;
  return dispatch(s.d, s.in_dtype, [&](auto dc, auto tc) {
    constexpr int D = decltype(dc)::value;
    using T = decltype(tc);
    const int n_state = with_state ? s.Hv * (D / kRows) : 0;
    const int per_thread = 16 / (int)sizeof(T);
    const int n_hist = with_hist ? (s.C / per_thread + kScanThreads - 1) / kScanThreads : 0;
    dim3 grid(n_state + n_hist, s.B, s.n_layers);
    return launch_kernel(commit_kernel<D, T>, grid, dim3(kScanThreads), 0, st, pdl, s, t, lb, accepted, len, lmax, n_state);
  });
}

cudaError_t launch_path_from_node(const TreeDev& t, int B, int N, const int32_t* node, int lmax,
                                  int32_t* accepted, int32_t* len, int32_t* status, cudaStream_t st) {
  path_from_node_kernel<<<(B + 63) / 64, 64, 0, st>>>(t, B, N, node, lmax, accepted, len, status);
  return cudaGetLastError();
}

}  // namespace lumo
