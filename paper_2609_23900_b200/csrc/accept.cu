// Device-resident acceptance walk: accepted path, its length, the pending token and the final row
// as fixed-shape device products (paper Algorithm 1, "Select one continuation"; Sec. "One
// device-selected path drives native continuation"), so that verify -> select -> commit needs no
// host round trip.  One thread-block cluster per sequence (the vocabulary is split over its CTAs,
// partial results meet through distributed shared memory) walks from the pre-tree state through the
// children of the current node in ascending logical index.
//
//   greedy     accept the child whose token equals argmax of the current target row (lowest token
//              index on ties); otherwise stop, the pending token is that argmax.
//   rejection  child c with token x is accepted iff u_c q_c(x) Z < r(x), r the unnormalised residual
//              target (r = p at first) and Z its sum; a rejection replaces r by (r - Z q_c)+ (accepted
//              mass min(p, q), residual mass proportional to (p - q)+, Appendix "Serving configuration
//              and measurement"); when no child is accepted the pending token is drawn from r / Z by an
//              exponential race argmax_i r_i / e_i over caller-supplied Exp(1) variates.
// Decisions that turn floats into integers use fixed precisions: the acceptance test and the residual
// update in float64 (separate multiply and subtract, no contraction), the residual stored in float32,
// the race keys as correctly rounded float32 quotients; sums are float64 in a fixed order.
#include <cooperative_groups.h>
#include <cuda_runtime.h>

#include "internal.h"

namespace cg = cooperative_groups;

namespace lumo {

namespace {

constexpr int kAcceptThreads = 512;
constexpr int kAcceptCluster = 8;       // CTAs per sequence: the vocabulary is split over a cluster

// A CTA's partial result, read by its peers through distributed shared memory.
struct ClusterSlot { double sum; float val; int idx; int flag; };

// Visit this CTA's slice [lo, hi) of the vocabulary with kAcceptUnroll independent loads in flight per
// thread; each thread sees its indices in ascending order.
constexpr int kAcceptUnroll = 8;
template <class Load, class Use>
__device__ __forceinline__ void for_slice(int lo, int hi, Load load, Use use) {
  for (int base = lo + (int)threadIdx.x; base < hi; base += kAcceptUnroll * kAcceptThreads) {
    decltype(load(0)) vals[kAcceptUnroll];
#pragma unroll
    for (int k = 0; k < kAcceptUnroll; ++k) {
      const int i = base + k * kAcceptThreads;
      if (i < hi) vals[k] = load(i);
    }
#pragma unroll
    for (int k = 0; k < kAcceptUnroll; ++k) {
      const int i = base + k * kAcceptThreads;
      if (i < hi) use(i, vals[k]);
    }
  }
}

// Cluster-wide reductions.  Each CTA reduces its slice, publishes the partial in one of two alternating
// slots of its shared memory, and after one cluster barrier warp 0 of every CTA combines all partials
// with the same shuffle tree, so all CTAs reach bit-identical results and take the same branches.  The
// slot written in reduction k is next written in reduction k + 2, i.e. after the barrier of reduction
// k + 1, which no CTA passes before it has read slot k.
struct Exchange {
  double red[kAcceptThreads / 32];
  float redv[kAcceptThreads / 32];
  int redi[kAcceptThreads / 32];
  ClusterSlot slot[2];
  ClusterSlot result;
  int parity;
};

__device__ double cluster_sum(cg::cluster_group& cl, double v, Exchange* x) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if (lane == 0) x->red[warp] = v;
  __syncthreads();
  const int par = x->parity;
  if (warp == 0) {
    double t = lane < kAcceptThreads / 32 ? x->red[lane] : 0.0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (lane == 0) x->slot[par].sum = t;
  }
  cl.sync();
  if (warp == 0) {
    double t = lane < (int)cl.num_blocks() ? cl.map_shared_rank(&x->slot[par], lane)->sum : 0.0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (lane == 0) { x->result.sum = t; x->parity = par ^ 1; }
  }
  __syncthreads();
  return x->result.sum;
}

__device__ __forceinline__ void argmax_step(float& v, int& i, int o) {
  const float ov = __shfl_xor_sync(0xffffffffu, v, o);
  const int oi = __shfl_xor_sync(0xffffffffu, i, o);
  if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
}

// argmax with the lowest index on ties over the whole cluster; every thread returns the result
__device__ int cluster_argmax(cg::cluster_group& cl, float v, int i, Exchange* x) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) argmax_step(v, i, o);
  if (lane == 0) { x->redv[warp] = v; x->redi[warp] = i; }
  __syncthreads();
  const int par = x->parity;
  if (warp == 0) {
    float bv = lane < kAcceptThreads / 32 ? x->redv[lane] : -2.f;
    int bi = lane < kAcceptThreads / 32 ? x->redi[lane] : 0x7fffffff;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) argmax_step(bv, bi, o);
    if (lane == 0) { x->slot[par].val = bv; x->slot[par].idx = bi; }
  }
  cl.sync();
  if (warp == 0) {
    float bv = -2.f;
    int bi = 0x7fffffff;
    if (lane < (int)cl.num_blocks()) {
      const ClusterSlot* o = cl.map_shared_rank(&x->slot[par], lane);
      bv = o->val;
      bi = o->idx;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) argmax_step(bv, bi, o);
    if (lane == 0) { x->result.idx = bi; x->parity = par ^ 1; }
  }
  __syncthreads();
  return x->result.idx;
}

__global__ void __launch_bounds__(kAcceptThreads)
accept_kernel(TreeDev t, int N, int Ns, AcceptView a, int lmax, int32_t* __restrict__ accepted,
              int32_t* __restrict__ len_out, int32_t* __restrict__ next_token, int32_t* __restrict__ final_node) {
  // this sequence's tree, staged once: the walk's dependent lookups then stay on chip
  __shared__ int32_t parent_child_off[kMaxNodes + 2], child_list[kMaxNodes], slot_map[kMaxNodes], tok_of_node[kMaxNodes];
  __shared__ Exchange xch;
  cg::cluster_group cl = cg::this_cluster();
  const int rank = (int)cl.block_rank(), nblk = (int)cl.num_blocks();
  const int b = blockIdx.y, tid = threadIdx.x, V = a.V;
  // this CTA's slice of the vocabulary
  const int chunk = (V + nblk - 1) / nblk;
  const int v_lo = rank * chunk, v_hi = min(V, v_lo + chunk);
  for (int e = tid; e < N + 2; e += kAcceptThreads) parent_child_off[e] = t.child_off[(size_t)b * (N + 2) + e];
  for (int e = tid; e < N; e += kAcceptThreads) {
    child_list[e] = t.child_list[(size_t)b * N + e];
    const int row = t.slot[(size_t)b * N + e];
    slot_map[e] = row;
    tok_of_node[e] = a.token[(size_t)b * Ns + row];
  }
  if (tid == 0) xch.parity = 0;
  __syncthreads();
  float* r = a.work + (size_t)b * V;
  int32_t* acc = accepted + (size_t)b * lmax;
  if (rank == 0)
    for (int e = tid; e < lmax; e += kAcceptThreads) acc[e] = -1;
  int cur = -1, len = 0, nxt = 0;

  for (int step = 0; step <= lmax; ++step) {                 // bounded: a path has at most lmax nodes
    const int prow = cur < 0 ? Ns : slot_map[cur];
    const float* p = a.p_target + ((size_t)b * (Ns + 1) + prow) * V;
    const int c_lo = parent_child_off[cur + 1], c_hi = parent_child_off[cur + 2];
    int took = -1;
    if (a.mode == 0) {
      float bv = -1.f;
      int bi = 0x7fffffff;
      auto look = [&](int i, float v) { if (v > bv) { bv = v; bi = i; } };     // ascending i per thread
      if ((V & 3) == 0 && (reinterpret_cast<uintptr_t>(p) & 15) == 0) {
        // rows on 16-byte boundaries: the body of the slice in 16-byte loads, all of a thread's loads
        // of one round in flight together; ragged ends element by element
        const int a4 = (v_lo + 3) & ~3, b4 = max(a4, v_hi & ~3);
        constexpr int kU4 = 5;
        for (int q0 = a4 / 4 + tid; q0 < b4 / 4; q0 += kU4 * kAcceptThreads) {   // bounded: slice
          float4 vals[kU4];
#pragma unroll
          for (int k = 0; k < kU4; ++k) {
            const int q = q0 + k * kAcceptThreads;
            if (q < b4 / 4) vals[k] = *reinterpret_cast<const float4*>(p + 4 * (size_t)q);
          }
#pragma unroll
          for (int k = 0; k < kU4; ++k) {
            const int q = q0 + k * kAcceptThreads;
            if (q < b4 / 4) { look(4 * q, vals[k].x); look(4 * q + 1, vals[k].y); look(4 * q + 2, vals[k].z); look(4 * q + 3, vals[k].w); }
          }
        }
        // the ragged ends hold lower (head) or higher (tail) indices than the body: ties are settled
        // by index in the reduction, and within a thread the head is visited last but compared with >
        // against a body value of higher index, so an equal head value must win explicitly
        for (int i = v_lo + tid; i < min(a4, v_hi); i += kAcceptThreads) { const float v = p[i]; if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; } }
        for (int i = b4 + tid; i < v_hi; i += kAcceptThreads) look(i, p[i]);
      } else {
        for_slice(v_lo, v_hi, [&](int i) { return p[i]; }, look);
      }
      nxt = cluster_argmax(cl, bv, bi, &xch);
      if (len < lmax)
        for (int ci = c_lo; ci < c_hi; ++ci) {                // bounded: children of one node
          const int c = child_list[ci];
          if (tok_of_node[c] == nxt) { took = c; break; }
        }
    } else {
      double zp = 0.0;
      for_slice(v_lo, v_hi, [&](int i) { return p[i]; }, [&](int i, float v) { r[i] = v; zp += (double)v; });
      double Z = cluster_sum(cl, zp, &xch);            // its cluster barriers also publish r
      for (int ci = c_lo; ci < c_hi && len < lmax; ++ci) {    // bounded: children of one node
        const int c = child_list[ci];
        const int sc = slot_map[c];
        const int x = tok_of_node[c];
        const float* q = a.q_draft + ((size_t)b * Ns + sc) * V;
        // every CTA evaluates the same test on the same values (r[x] was published by a cluster barrier)
        const double lhs = __dmul_rn(__dmul_rn((double)a.uniforms[(size_t)b * Ns + sc], (double)q[x]), Z);
        const float rx = *reinterpret_cast<volatile const float*>(r + x);
        cl.sync();                                             // everyone has read r[x] before it changes
        if (lhs < (double)rx) { took = c; break; }
        double zn = 0.0;
        for_slice(v_lo, v_hi, [&](int i) { return make_float2(r[i], q[i]); },
                  [&](int i, float2 rq) {
                    const double d = __dsub_rn((double)rq.x, __dmul_rn(Z, (double)rq.y));
                    const float rn = (float)(d > 0.0 ? d : 0.0);
                    r[i] = rn;
                    zn += (double)rn;
                  });
        const double Zn = cluster_sum(cl, zn, &xch);
        if (Zn > 0.0) Z = Zn;
        else {                                                 // empty residual: restore the target row
          double z2 = 0.0;
          for_slice(v_lo, v_hi, [&](int i) { return p[i]; }, [&](int i, float v) { r[i] = v; z2 += (double)v; });
          Z = cluster_sum(cl, z2, &xch);
        }
      }
      if (took < 0) {                                          // draw the pending token from r / Z
        const float* noise = a.noise + (size_t)b * V;
        float bv = -1.f;
        int bi = 0x7fffffff;
        for_slice(v_lo, v_hi, [&](int i) { return make_float2(r[i], noise[i]); },   // own slice of r
                  [&](int i, float2 rn) {
                    const float key = __fdiv_rn(rn.x, rn.y);
                    if (key > bv) { bv = key; bi = i; }
                  });
        nxt = cluster_argmax(cl, bv, bi, &xch);
      }
    }
    if (took < 0) break;                                       // uniform over the cluster
    if (rank == 0 && tid == 0) acc[len] = took;
    cur = took;
    ++len;
  }
  if (rank == 0 && tid == 0) { len_out[b] = len; next_token[b] = nxt; final_node[b] = cur; }
  cl.sync();                                                   // no CTA leaves while a peer may still read its slots
}

}  // namespace

cudaError_t launch_accept(const TreeDev& t, int B, int N, int Ns, const AcceptView& a, int lmax, int32_t* accepted,
                          int32_t* len, int32_t* next_token, int32_t* final_node, cudaStream_t st) {
  static int cache[64] = {};
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int cluster = max_cluster_ctas(accept_kernel, kAcceptThreads, cache);
  if (cluster > kAcceptCluster && B * cluster > sms) cluster = kAcceptCluster;   // many sequences: smaller clusters
  while (cluster > 1 && a.V < cluster * kAcceptThreads) cluster >>= 1;           // small vocabularies
  return launch_cluster_kernel(accept_kernel, dim3(cluster, B), dim3(kAcceptThreads), cluster, st, t, N, Ns, a, lmax,
                               accepted, len, next_token, final_node);
}

}  // namespace lumo
