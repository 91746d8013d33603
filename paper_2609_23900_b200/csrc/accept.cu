// Device-resident acceptance walk: accepted path, its length, the pending token and the final row
// as fixed-shape device products (paper Algorithm 1, "Select one continuation"; Sec. "One
// device-selected path drives native continuation"), so that verify -> select -> commit needs no
// host round trip.  One CTA per sequence walks from the pre-tree state through the children of the
// current node in ascending logical index.
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
#include <cuda_runtime.h>

#include "internal.h"

namespace lumo {

namespace {

constexpr int kAcceptThreads = 512;

__device__ double block_sum(double v, double* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
  __syncthreads();                       // red may still be read from the previous reduction
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  double t = 0.0;
  for (int w = 0; w < kAcceptThreads / 32; ++w) t += red[w];     // fixed order, every thread the same
  return t;
}

// argmax with the lowest index on ties; every thread returns the result
__device__ int block_argmax(float v, int i, float* redv, int* redi) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_down_sync(0xffffffffu, v, o);
    const int oi = __shfl_down_sync(0xffffffffu, i, o);
    if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
  }
  __syncthreads();
  if ((threadIdx.x & 31) == 0) { redv[threadIdx.x >> 5] = v; redi[threadIdx.x >> 5] = i; }
  __syncthreads();
  float bv = redv[0];
  int bi = redi[0];
  for (int w = 1; w < kAcceptThreads / 32; ++w)
    if (redv[w] > bv || (redv[w] == bv && redi[w] < bi)) { bv = redv[w]; bi = redi[w]; }
  return bi;
}

__global__ void __launch_bounds__(kAcceptThreads)
accept_kernel(TreeDev t, int N, int Ns, AcceptView a, int lmax, int32_t* __restrict__ accepted,
              int32_t* __restrict__ len_out, int32_t* __restrict__ next_token, int32_t* __restrict__ final_node) {
  __shared__ double red[kAcceptThreads / 32];
  __shared__ float redv[kAcceptThreads / 32];
  __shared__ int redi[kAcceptThreads / 32];
  __shared__ int s_take;
  const int b = blockIdx.x, tid = threadIdx.x, V = a.V;
  const int32_t* parent_child_off = t.child_off + (size_t)b * (N + 2);
  const int32_t* child_list = t.child_list + (size_t)b * N;
  const int32_t* slot = t.slot + (size_t)b * N;
  const int32_t* token = a.token + (size_t)b * Ns;
  float* r = a.work + (size_t)b * V;
  int32_t* acc = accepted + (size_t)b * lmax;
  for (int e = tid; e < lmax; e += kAcceptThreads) acc[e] = -1;
  int cur = -1, len = 0, nxt = 0;

  for (int step = 0; step <= lmax; ++step) {                 // bounded: a path has at most lmax nodes
    const int prow = cur < 0 ? Ns : slot[cur];
    const float* p = a.p_target + ((size_t)b * (Ns + 1) + prow) * V;
    const int c_lo = parent_child_off[cur + 1], c_hi = parent_child_off[cur + 2];
    int took = -1;
    if (a.mode == 0) {
      float bv = -1.f;
      int bi = 0x7fffffff;
      for (int i = tid; i < V; i += kAcceptThreads) {         // strided, ascending per thread
        const float v = p[i];
        if (v > bv) { bv = v; bi = i; }
      }
      nxt = block_argmax(bv, bi, redv, redi);
      if (len < lmax)
        for (int ci = c_lo; ci < c_hi; ++ci) {                // bounded: children of one node
          const int c = child_list[ci];
          if (token[slot[c]] == nxt) { took = c; break; }
        }
    } else {
      double zp = 0.0;
      for (int i = tid; i < V; i += kAcceptThreads) { const float v = p[i]; r[i] = v; zp += (double)v; }
      double Z = block_sum(zp, red);
      for (int ci = c_lo; ci < c_hi && len < lmax; ++ci) {    // bounded: children of one node
        const int c = child_list[ci];
        const int sc = slot[c];
        const int x = token[sc];
        const float* q = a.q_draft + ((size_t)b * Ns + sc) * V;
        __syncthreads();                                       // r is complete
        if (tid == 0) {
          const double lhs = __dmul_rn(__dmul_rn((double)a.uniforms[(size_t)b * Ns + sc], (double)q[x]), Z);
          s_take = lhs < (double)r[x];
        }
        __syncthreads();
        if (s_take) { took = c; break; }
        double zn = 0.0;
        for (int i = tid; i < V; i += kAcceptThreads) {
          const double d = __dsub_rn((double)r[i], __dmul_rn(Z, (double)q[i]));
          const float rn = (float)(d > 0.0 ? d : 0.0);
          r[i] = rn;
          zn += (double)rn;
        }
        const double Zn = block_sum(zn, red);
        if (Zn > 0.0) Z = Zn;
        else {                                                 // empty residual: restore the target row
          double z2 = 0.0;
          for (int i = tid; i < V; i += kAcceptThreads) { const float v = p[i]; r[i] = v; z2 += (double)v; }
          Z = block_sum(z2, red);
        }
      }
      if (took < 0) {                                          // draw the pending token from r / Z
        __syncthreads();
        const float* noise = a.noise + (size_t)b * V;
        float bv = -1.f;
        int bi = 0x7fffffff;
        for (int i = tid; i < V; i += kAcceptThreads) {
          const float key = __fdiv_rn(r[i], noise[i]);
          if (key > bv) { bv = key; bi = i; }
        }
        nxt = block_argmax(bv, bi, redv, redi);
      }
    }
    if (took < 0) break;                                       // uniform over the CTA
    if (tid == 0) acc[len] = took;
    cur = took;
    ++len;
  }
  if (tid == 0) { len_out[b] = len; next_token[b] = nxt; final_node[b] = cur; }
}

}  // namespace

cudaError_t launch_accept(const TreeDev& t, int B, int N, int Ns, const AcceptView& a, int lmax, int32_t* accepted,
                          int32_t* len, int32_t* next_token, int32_t* final_node, cudaStream_t st) {
  accept_kernel<<<B, kAcceptThreads, 0, st>>>(t, N, Ns, a, lmax, accepted, len, next_token, final_node);
  return cudaGetLastError();
}

}  // namespace lumo
