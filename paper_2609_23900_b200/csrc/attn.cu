// Ancestry-masked decode attention of the tree verifier on tcgen05 (sm_100a): paper Sec. "One slot map
// governs attention and publication" (grouped query heads share staged KV tiles; split-K context
// partitions) and Sec. "State and the execution boundary" (the visibility relation).
//
// tree_attn_kernel: persistent, warp-specialised, one CTA per SM.  The work is the list of 128-key tiles
// of all (sequence, KV head, 128-row query tile) units in order; a CTA takes a contiguous share of that
// list (or, with an explicit partition count, one partition of one unit), and every maximal piece of
// its share that lies in one unit is a SEGMENT: one flash-attention pass whose normalised output and
// base-2 log-sum-exp go to a scratch slot; attn_merge_kernel combines the slots of a unit in order.
// The query rows of all heads that share the KV head sit in one tile (row = head-in-group * N + node),
// so a staged key/value tile serves the whole group.
//
//   warps 0-1  producers: TMA loads (4-d tensor maps, 128-byte swizzle) of K tiles into one ring of three
//              32 KB stages and of V tiles into another, one mbarrier pair (full / empty) per stage; a K
//              stage is free as soon as its S product has completed, long before the V stage of that tile
//   warp 2     tensor-core issuer: S = Q K^T into one of two S buffers in tensor memory (M 128, N 128,
//              K 128), and O += P V (M 128, N 128, K 128; V is the MN-major B operand as it lies in
//              memory) into a 128-column accumulator that stays in tensor memory for the whole segment;
//              the S products run two tiles ahead of the O products (a buffer is refilled as soon as the
//              softmax warps hold its logits in registers), so the softmax warps never wait for logits.  Both A operands (Q and P) live in tensor memory, so shared memory carries only the staged K and V tiles.  (Measured:
//              an N = 128 product issues at the tensor core's full rate, an N = 64 one at 70 % of it.)
//   warps 3-10 softmax: a query row (= tensor-memory lane) is shared by two threads (warps w and w + 4),
//              64 keys each.  A thread reads its logits, applies visibility by selection (never by
//              arithmetic on a masked logit), exponentiates against a REFERENCE maximum m, rounds to bf16
//              and stores P as the next A operand.  m is the row maximum of the first
//              tile and moves only when a later maximum exceeds it by more than 2^16; only then is the
//              accumulator rescaled in tensor memory (probabilities up to 2^16 are harmless: bf16 and fp32
//              share their exponent range).  The two threads of a row exchange their tile maxima through
//              shared memory and a 64-thread named barrier, so both take the same decision.  At the end of
//              a segment each reads its 64 columns of O, divides by the row sum and writes the slot.
//
// Only tiles that reach past the committed context need a mask; the mask of node i over the physical
// suffix is a bit row built with the tree descriptor.  Value rows of positions nobody may read (padding
// slots, beyond the suffix) are zeroed in the staged tile before the product, so that bytes outside the
// visible set cannot reach any output (0 x NaN).
//
// Every wait is bounded; a wait that runs out marks the sequence LUMO_SEQ_TIMEOUT, later waits of that
// thread are skipped, and every role still runs its (bounded) loops to the common exit, where tensor
// memory is freed.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "internal.h"

namespace lumo {

namespace {

constexpr int kDh = 128;
constexpr int kRows = 128;            // query rows per unit = tensor-memory lanes
constexpr int kKeys = 128;            // keys per tile
constexpr int kSoftmaxWarps = 8;
constexpr int kFirstSoftmaxWarp = 3;
constexpr int kThreads = 32 * (kFirstSoftmaxWarp + kSoftmaxWarps);   // K producer, V producer, issuer, eight softmax warps
constexpr int kStages = 3;            // per ring (K tiles and V tiles have a ring each)
constexpr int kTmemCols = 512;        // S buffers: columns 0..127 and 128..255, O: 256..383, Q (bf16 pairs): 384..447,
                                      // P (bf16 pairs): 448..511
constexpr int kColO = 256;
constexpr int kColQ = 384;
constexpr int kColP = 448;
constexpr int kSeqCache = 64;         // sequences whose context length, cache row and tile count are kept in shared memory
constexpr int kUnitCost = 5;          // what starting a unit costs a CTA (read-out of the one before, new queries, refill of
                                      // the pipeline: ~8 us measured), in tiles: the shares are evened out in these terms
constexpr int kMinTilesPerCta = 4;    // automatic mode: do not cut the work finer than this
constexpr float kRescaleStep = 16.f;  // the reference maximum moves when exceeded by more than this (log2 units)
constexpr uint32_t kSpinLimit = 1u << 24;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// shared memory map; the dynamic segment starts at offset 0 of the CTA's window (no static shared
// variables in this kernel), which the 128-byte swizzle needs 1024-aligned; checked at run time
constexpr int kHalfBytes = 16384;     // one dh half of a tile: [128 keys x 128 B]
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr int kOffK = 0;              // K ring
constexpr int kOffV = kStages * kTileBytes;
constexpr int kOffSmall = 2 * kStages * kTileBytes;   // 196608
struct Small {
  unsigned long long k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  unsigned long long s_full[2], s_read[2], p_full;
  unsigned long long q_full, o_free;
  unsigned long long q_req;           // the first segment's query loads have been issued (the rings may fill behind them)
  uint32_t tmem_base;
  uint32_t timed_out;
  int seq_ctx[kSeqCache], seq_row[kSeqCache], seq_nt[kSeqCache];   // ctx_len, cache_row and tile count of the first sequences
  float xchg[2][2][kRows];           // [tile parity][key half][row]: row maxima (and row sums at a segment's end)
};
constexpr int kSmemBytes = kOffSmall + 3584;
static_assert(sizeof(Small) <= 3584, "small block");
static_assert(kSmemBytes + 1024 <= 227 * 1024, "one CTA per SM");

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


// Same bounded wait without acquire semantics: for waits that are followed by tensor-memory accesses only,
// which tcgen05.fence::after_thread_sync orders (the default acquire form measured ~200 cycles even on a
// completed phase).
__device__ __forceinline__ bool mbar_wait_relaxed(unsigned long long* bar, uint32_t parity) {
  const uint32_t addr = smem_u32(bar);
  for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
    uint32_t done;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.relaxed.cta.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(done) : "r"(addr), "r"(parity) : "memory");
    if (done) return true;
  }
  return false;
}

// One box of a 4-d tiled tensor map (dh, KV head, position, cache row) into shared memory; completion
// is counted in bytes on `bar`.  c0 is 0 or 64 elements: a multiple of 16 bytes.
// The keys and values stream through once: they carry an evict-first L2 policy, so that what is reused across
// tiles and launches (queries, partial results, tables, the kernel's own instructions) stays in L2.
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, unsigned long long* bar, int c0, int c1,
                                            int c2, int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;\n"
      ::"r"(dst), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(p));
  return p;
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
// same product with the A operand in tensor memory (row = lane, two bf16 per 32-bit column, K-major)
__device__ __forceinline__ void umma_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&t);
}

__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }

// ---- work decomposition ----------------------------------------------------------------
// Units are numbered u = (b * Hkv + hkv) * RT + rt; unit u owns nt(b) tiles (0 for a sequence that fails
// its check).  Automatic mode: the units are laid end to end on a line, each preceded by kUnitCost idle
// positions (the price of starting it); CTA c owns the positions [c * per, (c + 1) * per), works on the tiles
// among them, and the slot of a segment is u + c (strictly increasing along the line, so unique).  Fixed mode (S partitions):
// CTA c owns partition c mod S of unit c / S, slot c.
struct Segment {
  int b, hkv, rt;     // unit
  int t0, n;          // first tile within the unit, tile count (n = 0 possible in fixed mode)
  int slot;
  int unit, slot0, nslots;   // the unit, and the slots all its segments write (ascending along the key range)
  int ctx, crow;
};

struct Work {
  const AttnArgs& a;
  const Small& sm;
  int b, q;           // current sequence, unit within the sequence
  int g, g_end;       // next position on the line, end of this CTA's share (the host bounds the line below 2^31)
  int g_unit;         // position at which the current unit's stretch (idle prefix, then its tiles) starts
  int nt;             // tiles per unit of the current sequence
  int per;            // automatic mode: positions per CTA
  bool fixed_done;

  __device__ __forceinline__ int tiles_of(const AttnArgs& a, int bb, int* ctx, int* crow) const {
    if (bb < kSeqCache) { *ctx = sm.seq_ctx[bb]; *crow = sm.seq_row[bb]; return sm.seq_nt[bb]; }
    *ctx = a.ctx_len[bb];
    *crow = a.cache_row[bb];
    if (seq_check(*ctx, *crow, a.Ns, a.n_rows, a.max_pos) != LUMO_SEQ_OK) return 0;
    return (*ctx + a.Ns + kKeys - 1) / kKeys;
  }

  __device__ __forceinline__ void init() {
    b = 0; q = 0; g = 0; g_end = 0; g_unit = 0; nt = 0; per = 1; fixed_done = false;
    if (a.S > 0) return;
    const int upb = a.Hkv * a.RT;       // units per sequence
    int total = 0;
    int cx, cr;
    for (int bb = 0; bb < a.B; ++bb) {
      const int n = tiles_of(a, bb, &cx, &cr);
      if (n > 0) total += (n + kUnitCost) * upb;
    }
    per = (total + (int)gridDim.x - 1) / (int)gridDim.x;
    if (per < kMinTilesPerCta) per = kMinTilesPerCta;
    g = (int)blockIdx.x * per;
    g_end = g + per < total ? g + per : total;
    // the unit whose stretch holds position g
    int acc = 0;
    for (b = 0; b < a.B; ++b) {
      nt = tiles_of(a, b, &cx, &cr);
      const int span = nt > 0 ? (nt + kUnitCost) * upb : 0;
      if (g < acc + span) { q = (g - acc) / (nt + kUnitCost); g_unit = acc + q * (nt + kUnitCost); break; }
      acc += span;
    }
  }

  __device__ Work(const AttnArgs& args, const Small& small) : a(args), sm(small) { init(); }

  // next segment of this CTA; false when the share is exhausted
  __device__ __forceinline__ bool next(Segment* s) {
    const int upb = a.Hkv * a.RT;
    if (a.S > 0) {
      if (fixed_done) return false;
      fixed_done = true;
      const int u = blockIdx.x / a.S, part = blockIdx.x - u * a.S;
      s->b = u / upb;
      const int r = u - s->b * upb;
      s->hkv = r / a.RT; s->rt = r - s->hkv * a.RT;
      const int n_all = tiles_of(a, s->b, &s->ctx, &s->crow);
      s->t0 = (int)(((long long)part * n_all) / a.S);
      s->n = (int)(((long long)(part + 1) * n_all) / a.S) - s->t0;
      s->slot = blockIdx.x;
      s->unit = u; s->slot0 = u * a.S; s->nslots = a.S;
      return n_all > 0;
    }
    while (g < g_end && b < a.B) {
      if (nt == 0 || g >= g_unit + nt + kUnitCost) {     // move to the next unit (skipping sequences without tiles)
        if (nt > 0) g_unit += nt + kUnitCost;
        if (nt == 0 || ++q == upb) {
          q = 0;
          int cx, cr;
          do { ++b; nt = b < a.B ? tiles_of(a, b, &cx, &cr) : 0; } while (b < a.B && nt == 0);
        }
        continue;
      }
      const int first = g_unit + kUnitCost;              // position of the unit's tile 0
      const int lo = g > first ? g : first;
      const int hi = first + nt < g_end ? first + nt : g_end;
      g = g_unit + nt + kUnitCost < g_end ? g_unit + nt + kUnitCost : g_end;
      if (lo >= hi) continue;                            // only idle positions of this unit fall into the share
      const int u = b * upb + q;
      s->b = b; s->hkv = q / a.RT; s->rt = q - s->hkv * a.RT;
      tiles_of(a, b, &s->ctx, &s->crow);
      s->t0 = lo - first;
      s->n = hi - lo;
      s->slot = u + blockIdx.x;
      s->unit = u;
      s->slot0 = u + first / per;
      s->nslots = (first + nt - 1) / per - first / per + 1;
      return true;
    }
    return false;
  }
};

__global__ void __launch_bounds__(kThreads, 1)
tree_attn_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, const AttnArgs a) {
  extern __shared__ __align__(1024) unsigned char smem[];
  Small& sm = *reinterpret_cast<Small*>(smem + kOffSmall);
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool aligned = (sbase & 1023u) == 0;   // cannot fail with this file's layout; refuse rather than mis-swizzle

  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&sm.tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.k_full[s], 1); mbar_init(&sm.k_empty[s], 1);
      mbar_init(&sm.v_full[s], 1); mbar_init(&sm.v_empty[s], 1);
    }
    mbar_init(&sm.s_full[0], 1);
    mbar_init(&sm.s_full[1], 1);
    mbar_init(&sm.s_read[0], kSoftmaxWarps);
    mbar_init(&sm.s_read[1], kSoftmaxWarps);
    mbar_init(&sm.p_full, kSoftmaxWarps);        // one arrival per softmax warp
    mbar_init(&sm.q_full, kSoftmaxWarps);
    mbar_init(&sm.q_req, kSoftmaxWarps);
    mbar_init(&sm.o_free, kSoftmaxWarps);
    sm.timed_out = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (tid < kSeqCache && tid < a.B) {          // the work iterator of every role reads these instead of global memory
    const int cx = a.ctx_len[tid], cr = a.cache_row[tid];
    sm.seq_ctx[tid] = cx; sm.seq_row[tid] = cr;
    sm.seq_nt[tid] = seq_check(cx, cr, a.Ns, a.n_rows, a.max_pos) == LUMO_SEQ_OK ? (cx + a.Ns + kKeys - 1) / kKeys : 0;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  Work work(a, sm);
  Segment sg;
  bool ok = aligned;
  uint32_t it = 0;        // tiles this CTA has started, over all segments: ring stage, S buffer and phases
  uint32_t nseg = 0;      // segments with tiles so far: phases of q_full and o_free

  if (warp < 2) {
    // ---------------- producers: warp 0 feeds the K ring, warp 1 the V ring ----------------
    if (lane == 0) {
      const bool is_v = warp == 1;
      const CUtensorMap* map = is_v ? &tm_v : &tm_k;
      unsigned long long* full = is_v ? sm.v_full : sm.k_full;
      unsigned long long* empty = is_v ? sm.v_empty : sm.k_empty;
      const uint32_t ring = sbase + (is_v ? kOffV : kOffK);
      const uint64_t stream_policy = l2_evict_first_policy();
      while (work.next(&sg)) {
        for (int j = 0; j < sg.n; ++j, ++it) {
          const uint32_t st = it % kStages, use = it / kStages;
          if (use > 0 && ok) ok = mbar_wait(&empty[st], (use - 1) & 1u);
          // Start-up: the rings of all CTAs fill at once (28 MB in flight) and the first segment's query rows
          // would queue behind them (measured: 3.4 us for 256 bytes per thread).  Only the first K tile goes
          // ahead of the queries; everything else waits until their loads have been issued (requests are served
          // roughly in order: the queries come back first, the rings fill behind them).
          if (it == (is_v ? 0u : 1u) && ok) ok = mbar_wait(&sm.q_req, 0);
          if (!ok) continue;
          mbar_expect_tx(&full[st], kTileBytes);
          const uint32_t dst = ring + st * kTileBytes;
          const int pos = (sg.t0 + j) * kKeys;
          // tensor-map dimensions ascend in stride: (dh, head, position, row) or (dh, position, head, row)
          const int c1 = a.layout ? pos : sg.hkv, c2 = a.layout ? sg.hkv : pos;
          tma_load_4d(dst, map, &full[st], 0, c1, c2, sg.crow, stream_policy);
          tma_load_4d(dst + kHalfBytes, map, &full[st], 64, c1, c2, sg.crow, stream_policy);
        }
      }
      if (!ok) sm.timed_out = 1u;
    }
  } else if (warp == 2) {
    // ---------------- tensor-core issuer ----------------
    if (lane == 0) {
      // S = Q K^T: A = Q in tensor memory, B = K tile (K-major: 128 key rows of 128 B per dh half).  Its
      // completion frees the K stage.
      auto issue_qk = [&](uint32_t t) {
        constexpr uint32_t id = umma_idesc(kRows, kKeys, 0, 0);
        const uint32_t kb = sbase + kOffK + (t % kStages) * kTileBytes;
        const uint32_t d = tmem + (t & 1u) * kKeys;
#pragma unroll
        for (int ks = 0; ks < kDh / 16; ++ks)
          umma_ta(d, tmem + kColQ + ks * 8, umma_desc(kb + (ks >> 2) * kHalfBytes + (ks & 3) * 32, 16, 1024), id, ks ? 1u : 0u);
        umma_commit(&sm.s_full[t & 1u]);
        umma_commit(&sm.k_empty[t % kStages]);
      };
      // O += P V: A = P in tensor memory, B = V tile as it lies in memory (MN-major: 128 B of dh per key
      // row, the two dh halves kHalfBytes apart, 16 keys = 2048 B per K step).  Its completion frees the
      // V stage and the P columns.
      auto issue_pv = [&](uint32_t t, bool first) {
        constexpr uint32_t id = umma_idesc(kRows, kDh, 0, 1);
        const uint32_t vb = sbase + kOffV + (t % kStages) * kTileBytes;
#pragma unroll
        for (int ks = 0; ks < kKeys / 16; ++ks)
          umma_ta(tmem + kColO, tmem + kColP + ks * 8, umma_desc(vb + ks * 2048, kHalfBytes, 1024), id, (first && ks == 0) ? 0u : 1u);
        umma_commit(&sm.v_empty[t % kStages]);
      };
      auto qk_when_ready = [&](uint32_t t) {
        if (ok) ok = mbar_wait(&sm.k_full[t % kStages], (t / kStages) & 1u);
        tc_fence_after();
        if (ok) issue_qk(t);
      };
      while (work.next(&sg)) {
        if (sg.n == 0) continue;
        if (ok) ok = mbar_wait(&sm.q_full, nseg & 1u);
        // the logits run two tiles ahead of the O products: S buffer t & 1 is free once the softmax warps
        // have turned tile t - 2 into P (their p_full arrival, awaited below)
        qk_when_ready(it);
        if (sg.n > 1) qk_when_ready(it + 1);
        for (int j = 0; j < sg.n; ++j, ++it) {
          // Two waits per tile, each followed by one product.  (An mbarrier wait between tensor-core
          // instructions costs this thread a few hundred cycles, measured; the waits for the TMA tiles are
          // therefore done by the first softmax warp before it arrives on these two barriers.)
          if (j + 2 < sg.n) {
            // the softmax warps hold tile it's logits in registers: its S buffer takes the logits of tile it + 2
            if (ok) ok = mbar_wait(&sm.s_read[it & 1u], (it >> 1) & 1u);
            tc_fence_after();
            if (ok) issue_qk(it + 2);
          }
          if (ok) ok = mbar_wait(&sm.p_full, it & 1u);
          if (j == 0 && nseg > 0 && ok) ok = mbar_wait(&sm.o_free, (nseg - 1) & 1u);
          tc_fence_after();
          if (ok) issue_pv(it, j == 0);
        }
        ++nseg;
      }
      if (!ok) sm.timed_out = 1u;
    }
  } else {
    // ---------------- softmax warps ----------------
    // Warps w and w + 4 share the 32 rows of one lane quarter; the first takes keys 0..63 of every tile
    // and output columns 0..63, the second the other halves.
    const int sw = warp - kFirstSoftmaxWarp;     // 0..7
    const int half = sw >> 2;
    const int row = 32 * (warp & 3) + lane;      // tensor-memory lane this warp may touch
    const int sthread = tid - 32 * kFirstSoftmaxWarp;   // 0..255
    const uint32_t tmem_lane = tmem + ((uint32_t)(32 * (warp & 3)) << 16);
    const int pair_bar = 1 + (warp & 3);         // named barrier of the two warps of a lane quarter
    const float sl2 = a.scale_log2;
    const int GN = a.G * a.N;
    // Query tile of a segment into tensor memory: this thread's half of its row, two bf16 per column (zeros
    // beyond the group); then one arrival per warp on q_full.  Called when the S products of the segment before
    // have all completed (every thread awaited their s_full phases): for the first segment at once, for the
    // others right after the last tile's probabilities have been handed over, BEFORE that segment's read-out,
    // so that the next logits are computed while the accumulator is being written out.
    auto store_q = [&](const Segment& g) {
      const int rgq = g.rt * kRows + row;
      const bool okq = rgq < GN;
      const int hq = okq ? rgq / a.N : 0, nq = okq ? rgq - hq * a.N : 0;
      const uint4* qrow = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(a.q) +
                                                         (((size_t)g.b * a.N + nq) * a.Hq + (size_t)g.hkv * a.G + hq) * kDh);
      uint32_t qr[32];
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint4 v = okq ? __ldg(qrow + half * 8 + c) : make_uint4(0u, 0u, 0u, 0u);
        qr[4 * c] = v.x; qr[4 * c + 1] = v.y; qr[4 * c + 2] = v.z; qr[4 * c + 3] = v.w;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.q_req);     // every lane's loads are on their way
      tmem_st32(tmem_lane + kColQ + half * 32, qr);
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.q_full);
    };
    Segment sgn;
    bool have = work.next(&sg);
    if (have && sg.n > 0) store_q(sg);
    for (; have; sg = sgn) {
      const int rg = sg.rt * kRows + row;
      const bool row_ok = rg < GN;
      const int hl = row_ok ? rg / a.N : 0, node = row_ok ? rg - hl * a.N : 0;
      // a slot holds its rows by groups of four columns, [column group][row][4]: the 32 lanes of a store (32
      // rows, one group) write 512 contiguous bytes, and the merge kernel reads them the same way
      float4* slot_o = reinterpret_cast<float4*>(a.part_o + (size_t)sg.slot * kRows * kDh) + (size_t)(half * 16) * kRows + row;
      float* slot_l = a.part_lse + (size_t)sg.slot * kRows + row;
      if (sthread == 0) a.unit_slots[sg.unit] = make_int2(sg.slot0, sg.nslots);   // for the merge (same pair from every writer)
      if (sg.n == 0) {                           // empty partition (fixed mode): an empty slot
        if (row_ok) {
          for (int e = 0; e < 16; ++e) slot_o[(size_t)e * kRows] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (half == 0) *slot_l = -INFINITY;
        }
        have = work.next(&sgn);                  // (an empty partition is a CTA's only segment)
        if (have && sgn.n > 0) store_q(sgn);
        continue;
      }
      const uint32_t* visw = a.vis + ((size_t)sg.b * a.N + node) * 8;
      const uint32_t* usedw = a.used + (size_t)sg.b * 8;
      float m = -INFINITY, l = 0.f;              // reference maximum (log2 units), this thread's part of the row sum
      for (int j = 0; j < sg.n; ++j, ++it) {
        const uint32_t buf = it & 1u;
        const int kpos0 = (sg.t0 + j) * kKeys + half * 64;   // first key of this thread's 64
        const bool tail = (sg.t0 + j + 1) * kKeys > sg.ctx;  // uniform: the tile reaches past the committed context
        unsigned long long vm = ~0ull;
        if (tail) {
          vm = 0ull;
          for (int c = 0; c < 64; ++c) {
            const int p = kpos0 + c;
            bool v = p < sg.ctx;
            if (!v) {
              const int s = p - sg.ctx;
              if (s < a.Ns) v = (__ldg(visw + (s >> 5)) >> (s & 31)) & 1u;
            }
            vm |= (unsigned long long)v << c;
          }
        }
        if (ok) ok = mbar_wait_relaxed(&sm.s_full[buf], (it >> 1) & 1u);
        tc_fence_after();
        __syncwarp();
        uint32_t sr[64];
        tmem_ld32(tmem_lane + buf * kKeys + half * 64, sr);
        tmem_ld32(tmem_lane + buf * kKeys + half * 64 + 32, sr + 32);
        tmem_ld_wait();
        // the logits are in registers: the S buffer may take the logits of tile it + 2 (whose keys must have landed)
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (sw == 0 && j + 2 < sg.n && ok) ok = mbar_wait(&sm.k_full[(it + 2) % kStages], ((it + 2) / kStages) & 1u);
          mbar_arrive(&sm.s_read[buf]);
        }
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        if (!tail) {
#pragma unroll
          for (int e = 0; e < 64; ++e) mx4[e & 3] = fmaxf(mx4[e & 3], __uint_as_float(sr[e]));
        } else {
#pragma unroll
          for (int e = 0; e < 64; ++e) mx4[e & 3] = fmaxf(mx4[e & 3], ((vm >> e) & 1ull) ? __uint_as_float(sr[e]) : -INFINITY);
        }
        float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sl2;
        // the row maximum of the tile: exchange with the thread that holds the other 64 keys
        sm.xchg[buf][half][row] = mx;
        asm volatile("bar.sync %0, 64;\n" ::"r"(pair_bar) : "memory");
        mx = fmaxf(mx, sm.xchg[buf][half ^ 1][row]);
        // reference maximum: set by the first tile that shows the row a key; moved (with a rescale of the
        // accumulator) only when exceeded by more than kRescaleStep.  Both threads of a row decide alike.
        float corr = 1.f;
        if (m == -INFINITY) m = mx;
        else if (mx > m + kRescaleStep) { corr = ex2(m - mx); m = mx; }
        if (__any_sync(0xffffffffu, corr != 1.f)) {
          // O still holds the products up to the previous tile: wait for them, then scale this thread's columns
          if (ok) ok = mbar_wait(&sm.v_empty[(it - 1) % kStages], ((it - 1) / kStages) & 1u);
          tc_fence_after();
          __syncwarp();
#pragma unroll 1
          for (int c = 0; c < 64; c += 32) {
            uint32_t orr[32];
            tmem_ld32(tmem_lane + kColO + half * 64 + c, orr);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) orr[e] = __float_as_uint(__uint_as_float(orr[e]) * corr);
            tmem_st32(tmem_lane + kColO + half * 64 + c, orr);
          }
          tmem_st_wait();
          l *= corr;
        }
        const float mu = m == -INFINITY ? 0.f : m;
        // P has columns of its own (32 per thread), free once the previous tile's O product has completed
        uint32_t pk[32];
        float ls4[4] = {0.f, 0.f, 0.f, 0.f};
        if (!tail) {
#pragma unroll
          for (int c = 0; c < 64; c += 2) {
            const float p0 = ex2(fmaf(__uint_as_float(sr[c]), sl2, -mu));
            const float p1 = ex2(fmaf(__uint_as_float(sr[c + 1]), sl2, -mu));
            ls4[(c >> 1) & 3] += p0 + p1;
            pk[c >> 1] = pack_bf16(p0, p1);
          }
        } else {
#pragma unroll
          for (int c = 0; c < 64; c += 2) {
            const float p0 = ((vm >> c) & 1ull) ? ex2(fmaf(__uint_as_float(sr[c]), sl2, -mu)) : 0.f;
            const float p1 = ((vm >> (c + 1)) & 1ull) ? ex2(fmaf(__uint_as_float(sr[c + 1]), sl2, -mu)) : 0.f;
            ls4[(c >> 1) & 3] += p0 + p1;
            pk[c >> 1] = pack_bf16(p0, p1);
          }
        }
        l += (ls4[0] + ls4[1]) + (ls4[2] + ls4[3]);
        if (it > 0 && ok) ok = mbar_wait_relaxed(&sm.v_empty[(it - 1) % kStages], ((it - 1) / kStages) & 1u);
        tc_fence_after();
        tmem_st32(tmem_lane + kColP + half * 32, pk);
        if (tail) {
          // value rows nobody may read: zero them in the staged tile (two 128-byte rows per key)
          const uint32_t st = it % kStages;
          if (ok) ok = mbar_wait(&sm.v_full[st], (it / kStages) & 1u);
          const int c = sthread >> 1, hh = sthread & 1;
          const int p = (sg.t0 + j) * kKeys + c;
          bool dead = false;
          if (p >= sg.ctx) {
            const int s = p - sg.ctx;
            dead = s >= a.Ns || !((__ldg(usedw + (s >> 5)) >> (s & 31)) & 1u);
          }
          if (dead) {
            uint4* vrow = reinterpret_cast<uint4*>(smem + kOffV + st * kTileBytes + hh * kHalfBytes + c * 128);
#pragma unroll
            for (int e = 0; e < 8; ++e) vrow[e] = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_async_proxy();                   // for the tensor core's reads
        }
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (sw == 0 && ok) ok = mbar_wait(&sm.v_full[it % kStages], (it / kStages) & 1u);   // on behalf of the issuer
          mbar_arrive(&sm.p_full);
        }
      }
      // end of the segment.  First the next segment's queries (its logits then run under this read-out) ...
      have = work.next(&sgn);
      if (have && sgn.n > 0) store_q(sgn);
      // ... then the last O product, normalise and write the slot
      if (ok) ok = mbar_wait(&sm.v_empty[(it - 1) % kStages], ((it - 1) / kStages) & 1u);
      tc_fence_after();
      sm.xchg[0][half][row] = l;
      asm volatile("bar.sync %0, 64;\n" ::"r"(pair_bar) : "memory");
      const float lt = sm.xchg[0][0][row] + sm.xchg[0][1][row];
      const float inv = lt > 0.f ? 1.f / lt : 0.f;
#pragma unroll 1
      for (int c = 0; c < 64; c += 32) {
        uint32_t orr[32];
        tmem_ld32(tmem_lane + kColO + half * 64 + c, orr);
        tmem_ld_wait();
        if (row_ok) {
#pragma unroll
          for (int e = 0; e < 32; e += 4)
            slot_o[(size_t)((c + e) >> 2) * kRows] =
                make_float4(__uint_as_float(orr[e]) * inv, __uint_as_float(orr[e + 1]) * inv,
                            __uint_as_float(orr[e + 2]) * inv, __uint_as_float(orr[e + 3]) * inv);
        }
      }
      if (row_ok && half == 0) *slot_l = lt > 0.f ? m + log2f(lt) : -INFINITY;
      tc_fence_before();
      asm volatile("bar.sync %0, 64;\n" ::"r"(pair_bar) : "memory");   // the partner has read xchg[0] before the next segment writes it
      if (lane == 0) mbar_arrive(&sm.o_free);
      ++nseg;
    }
    if (!ok) sm.timed_out = 1u;
  }

  tc_fence_before();
  __syncthreads();
  if (sm.timed_out && tid == 0) *a.fail_flag = a.launch_id;   // the merge kernel turns this into status words
  if (warp == 2) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

// Combination of a unit's slots: a warp takes 32 rows of a unit and one group of four columns (the slots
// hold [column group][row][4], so its loads are contiguous), a lane one row; slots in order (so the result
// for a given decomposition is reproducible), weights exp2(lse_s - max lse).
// kBatch: slots per flight of loads (8: few slots per unit and a small register footprint, so that the CTAs
// are staged beside the draining attention kernel; 24: a unit spread over all SMs, about 19 slots at batch 1)
template <int kBatch>
__global__ void __launch_bounds__(256) attn_merge_kernel(const AttnArgs a) {
  pdl_wait();          // launched as a programmatic dependent of the attention kernel: its slots are complete from here on
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int GN = a.G * a.N;
  const int upb = a.Hkv * a.RT;
  const long long w = (long long)blockIdx.x * 8 + warp;
  if (w >= (long long)a.B * upb * 128) return;
  const int cg = (int)(w & 31), rq = (int)((w >> 5) & 3);
  const int u = (int)(w >> 7);
  const int b = u / upb;
  const int rem = u - b * upb;
  const int hkv = rem / a.RT, rt = rem - hkv * a.RT;
  const int r = rq * 32 + lane;
  const int rg = rt * kRows + r;
  // Three independent loads first (one round trip): the sequence's context length and cache row, and the slot
  // range the attention kernel recorded for this unit (meaningless for a sequence that fails its check).
  const int cx = a.ctx_len[b], cr = a.cache_row[b];
  const int2 t = a.unit_slots[u];
  const int st = seq_check(cx, cr, a.Ns, a.n_rows, a.max_pos);
  // status word of the sequence: its check, else whether any wait of this launch's attention kernel ran out
  // (then the outputs of the whole call are suspect)
  if (a.status && lane == 0 && rem == 0 && rq == 0 && cg == 0)
    a.status[b] = st != LUMO_SEQ_OK ? st : (*a.fail_flag == a.launch_id ? (int)LUMO_SEQ_TIMEOUT : (int)LUMO_SEQ_OK);
  if (rg >= GN) return;                      // rows beyond the group (no warp-wide operation follows)
  const int hl = rg / a.N, node = rg - hl * a.N;
  const size_t out_row = (((size_t)b * a.N + node) * a.Hq + (size_t)hkv * a.G + hl);
  float4* dst = reinterpret_cast<float4*>(a.out + out_row * kDh) + cg;
  if (st != LUMO_SEQ_OK) {                   // the sequence owns no tiles: zeros
    *dst = make_float4(0.f, 0.f, 0.f, 0.f);
    if (a.lse && cg == 0) a.lse[out_row] = 0.f;
    return;
  }
  const int slot0 = t.x, nslot = t.y;
  const float* lse_p = a.part_lse + (size_t)slot0 * kRows + r;                          // + slot * kRows
  const float4* row_p = reinterpret_cast<const float4*>(a.part_o) + ((size_t)slot0 * 32 + cg) * kRows + r;   // + slot * 32 * kRows
  // Second round trip: the rows of the first kBatch slots together with all log-sum-exps; further slots follow
  // kBatch at a time.  The combination runs in slot order against the maximum of all log-sum-exps, whatever the
  // grouping of the loads.
  float4 v[kBatch];
  float ls[kBatch];
  auto load_batch = [&](int s0) {
#pragma unroll
    for (int k = 0; k < kBatch; ++k) {
      const bool in = s0 + k < nslot;
      ls[k] = in ? lse_p[(size_t)(s0 + k) * kRows] : -INFINITY;
      v[k] = in ? row_p[(size_t)(s0 + k) * 32 * kRows] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  load_batch(0);
  float mx = -INFINITY;
#pragma unroll
  for (int k = 0; k < kBatch; ++k) mx = fmaxf(mx, ls[k]);
  for (int sl = kBatch; sl < nslot; ++sl) mx = fmaxf(mx, lse_p[(size_t)sl * kRows]);   // bounded: < 256 slots
  float den = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s0 = 0; s0 < nslot; s0 += kBatch) {
    if (s0) load_batch(s0);
#pragma unroll
    for (int k = 0; k < kBatch; ++k) {
      if (ls[k] == -INFINITY) continue;      // none, or an empty slot
      const float wgt = ex2(ls[k] - mx);
      den += wgt;
      acc.x = fmaf(wgt, v[k].x, acc.x); acc.y = fmaf(wgt, v[k].y, acc.y);
      acc.z = fmaf(wgt, v[k].z, acc.z); acc.w = fmaf(wgt, v[k].w, acc.w);
    }
  }
  const float inv = den > 0.f ? 1.f / den : 0.f;
  *dst = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
  if (a.lse && cg == 0) a.lse[out_row] = den > 0.f ? (mx + log2f(den)) * kLn2 : -INFINITY;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map of one cache: dims (dh, KV head, position, row), box 64 x 1 x 64 x 1, 128-byte swizzle;
// positions beyond max_positions read as zeros.
cudaError_t encode_cache_map(void* cache, int Hkv, int max_pos, int n_rows, int layout, CUtensorMap* map, std::string* err) {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
    if (e != cudaSuccess) return e;
    if (q != cudaDriverEntryPointSuccess || !p) { *err = "the driver does not export cuTensorMapEncodeTiled"; return cudaErrorNotSupported; }
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  const cuuint64_t row_bytes = (cuuint64_t)max_pos * Hkv * kDh * 2;
  cuuint64_t dims[4] = {(cuuint64_t)kDh, (cuuint64_t)Hkv, (cuuint64_t)max_pos, (cuuint64_t)n_rows};
  cuuint64_t strides[3] = {(cuuint64_t)kDh * 2, (cuuint64_t)Hkv * kDh * 2, row_bytes};
  cuuint32_t box[4] = {64, 1, (cuuint32_t)kKeys, 1};   // 16 KB
  if (layout == 1) {   // a head's positions adjacent
    dims[1] = (cuuint64_t)max_pos; dims[2] = (cuuint64_t)Hkv;
    strides[1] = (cuuint64_t)max_pos * kDh * 2;
    box[1] = (cuuint32_t)kKeys; box[2] = 1;
  }
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, cache, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { *err = "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r); return cudaErrorInvalidValue; }
  return cudaSuccess;
}

}  // namespace

int attn_row_tiles(int G, int N) { return (G * N + kRows - 1) / kRows; }

// slots of partial results: automatic mode needs at most units + CTAs - 1, fixed mode units x partitions
size_t attn_units(const AttnShape& s) { return (size_t)s.B * s.Hkv * attn_row_tiles(s.Hq / s.Hkv, s.N); }

static size_t attn_slots(const AttnShape& s, int ctas) {
  const size_t units = (size_t)s.B * s.Hkv * attn_row_tiles(s.Hq / s.Hkv, s.N);
  return s.S > 0 ? units * s.S : units + ctas;
}

// 256 bytes whose first word says "a wait ran out in launch number ..." (at a fixed place, zero at allocation), then
// partial results [slots][128][128], their log-sum-exps [slots][128], the slot range of every unit [units][2]
size_t attn_scratch_bytes(const AttnShape& s, int sm_count) {
  return 256 + attn_slots(s, sm_count) * kRows * (kDh + 1) * sizeof(float) + attn_units(s) * sizeof(int2);
}

cudaError_t attn_plan(const AttnShape& s, const AttnLayerPtrs& p, const uint32_t* vis, const uint32_t* used, float* scratch,
                      int sm_count, uint32_t launch_id, AttnPlan* plan, std::string* err) {
  static bool configured[kMaxDevices] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < kMaxDevices && !configured[dev]) {
    e = cudaFuncSetAttribute(tree_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  e = encode_cache_map(p.k_cache, s.Hkv, s.max_pos, s.n_rows, s.layout, &plan->tk, err);
  if (e != cudaSuccess) return e;
  e = encode_cache_map(p.v_cache, s.Hkv, s.max_pos, s.n_rows, s.layout, &plan->tv, err);
  if (e != cudaSuccess) return e;
  AttnArgs& a = plan->a;
  a.q = p.q;
  a.out = p.out; a.lse = p.lse;
  a.G = s.Hq / s.Hkv; a.RT = attn_row_tiles(a.G, s.N); a.S = s.S;
  const size_t units = (size_t)s.B * s.Hkv * a.RT;
  a.C = s.S > 0 ? (int)(units * s.S) : sm_count;
  a.fail_flag = reinterpret_cast<uint32_t*>(scratch);
  scratch += 64;
  a.part_o = scratch;
  a.part_lse = scratch + attn_slots(s, sm_count) * kRows * kDh;
  a.unit_slots = reinterpret_cast<int2*>(a.part_lse + attn_slots(s, sm_count) * kRows);
  a.launch_id = launch_id;
  a.ctx_len = s.ctx_len; a.cache_row = s.cache_row; a.vis = vis; a.used = used; a.status = p.status;
  a.B = s.B; a.N = s.N; a.Ns = s.Ns; a.Hq = s.Hq; a.Hkv = s.Hkv; a.n_rows = s.n_rows; a.max_pos = s.max_pos;
  a.scale_log2 = s.scale * kLog2e;
  a.layout = s.layout;
  plan->grid = dim3(a.C, 1, 1);
  return cudaSuccess;
}

cudaError_t launch_attn(const AttnPlan& plan, cudaStream_t st) {
  tree_attn_kernel<<<plan.grid, kThreads, kSmemBytes, st>>>(plan.tk, plan.tv, plan.a);
  return cudaGetLastError();
}

cudaError_t launch_attn_merge(const AttnPlan& plan, cudaStream_t st) {
  // one warp per (unit, 32 rows, group of four columns): 128 warps per unit, 16 CTAs
  const long long ctas = (long long)plan.a.B * plan.a.Hkv * plan.a.RT * 16;
  // dependent launch: the CTAs are staged while the attention kernel drains and wait on the device for its end
  const long long units = (long long)plan.a.B * plan.a.Hkv * plan.a.RT;
  const long long slots_per_unit = plan.a.S > 0 ? plan.a.S : ((long long)plan.grid.x + units - 1) / units + 1;
  if (slots_per_unit > 12)
    return launch_kernel(attn_merge_kernel<24>, dim3((unsigned)ctas), dim3(256), 0, st, true, plan.a);
  return launch_kernel(attn_merge_kernel<8>, dim3((unsigned)ctas), dim3(256), 0, st, true, plan.a);
}

}  // namespace lumo
