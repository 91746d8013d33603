// KV-cache side of the attention half (sm_100a): the write of the tree's entries through the slot map and
// the re-linearisation of the accepted path at publication (paper Sec. "One slot map governs attention
// and publication"; Algorithm 1, "remap KV").  Pure data movement, bit-exact.
#include <cuda_runtime.h>

#include "internal.h"

namespace lumo {

namespace {

constexpr int kDh = 128;

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
  const int chunks = s.Hkv * kDh / 8;      // 16-byte chunks per entry (16 per head)
  const size_t src = ((size_t)b * s.N + i) * chunks;
  const uint4* kn = reinterpret_cast<const uint4*>(L.kn[l]) + src;
  const uint4* vn = reinterpret_cast<const uint4*>(L.vn[l]) + src;
  // chunk strides of the cache: position and head
  const size_t pos_st = s.layout ? 16 : (size_t)s.Hkv * 16, head_st = s.layout ? (size_t)s.max_pos * 16 : 16;
  const size_t dst = (size_t)crow * s.max_pos * chunks + (size_t)(ctx + s.slot[(size_t)b * s.N + i]) * pos_st;
  uint4* kc = reinterpret_cast<uint4*>(L.k[l]) + dst;
  uint4* vc = reinterpret_cast<uint4*>(L.v[l]) + dst;
  for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
    const size_t o = (size_t)(c >> 4) * head_st + (c & 15);
    kc[o] = __ldg(kn + c);
    vc[o] = __ldg(vn + c);
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
  const size_t pos_bytes = s.layout ? (size_t)kDh * 2 : (size_t)s.Hkv * kDh * 2;
  const size_t head_bytes = s.layout ? (size_t)s.max_pos * kDh * 2 : (size_t)kDh * 2;
  unsigned char* rowp = cache + (size_t)crow * s.max_pos * s.Hkv * kDh * 2 + (size_t)ctx * pos_bytes + (size_t)hkv * head_bytes;
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

}  // namespace

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
