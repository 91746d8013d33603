// Internal declarations shared by the host side and the kernels of liblumo_gdn.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>
#include <string>
#include <vector>

#include "lumo_gdn.h"

namespace lumo {

constexpr int kMaxNodes = 256;
constexpr int kMaxSlots = 1024;
constexpr int kMaxLayers = 64;
constexpr int kMaxAttnSlots = 256;                 // physical suffix the attention kernels take (8 mask words per node)
constexpr int kMaxAttnLayers = 32;
constexpr int kMaxDevices = 64;                    // per-device caches (kernel attributes, symbol addresses)
constexpr size_t kStaticStackBytes = 64u << 20;   // capacity of the built-in scan stack

// ---- scan schedule ------------------------------------------------------------------
// The scan kernel walks the whole tree depth first with the state tile of the current
// node's parent in registers.  An op is (kind << 24) | (flag << 20) | arg.
//   EMIT c          o_c from the parent's state (no state materialised); flag=1 also caches
//                   delta_c on chip for a later DESCEND c
//   EMIT_DESCEND c  EMIT c, then turn the registers into S_c in place
//   DESCEND c       turn the registers (S_parent) into S_c using the cached delta_c
//   PUSH l          save the registers to stack level l
//   POP l           restore the registers from stack level l; l = kPopRoot reloads the
//                   pre-tree state from the state pool
enum OpKind : int { OP_EMIT = 0, OP_EMIT_DESCEND = 1, OP_DESCEND = 2, OP_PUSH = 3, OP_POP = 4 };
constexpr int kPopRoot = 0xFFFF;
inline int make_op(int kind, int flag, int arg) { return (kind << 24) | (flag << 20) | (arg & 0xFFFF); }

struct HostTree {
  std::vector<int32_t> tab[LUMO_TAB_COUNT];
};

struct GramGroup {
  std::vector<int> nodes;    // logical ids ordered by (depth, index); every ancestor of a member is a member
  std::vector<char> emit;    // 1: this group writes the node's output
};

}  // namespace lumo

struct lumo_ctx {
  int device = 0;
  int sm_count = 0;
  std::string err;
  void* scratch = nullptr;      // scan stack levels
  size_t scratch_bytes = 0;
  void* attn_scratch = nullptr; // partial results of the attention partitions
  size_t attn_scratch_bytes = 0;
  uint32_t attn_launch_id = 0;
  // optional per-launch timing (lumo_ctx_timing_*): a fixed pool of event pairs
  int scan_algo = 0;            // 0 auto, 1 rank-1, 2 Gram form with forward substitution, 3 solved Gram form, 4 Gram form with closed-form tail, 5 the same with the output sum on the tensor core
  bool timeout_drill = false;   // test aid: the tensor-core scan skips its tensor-core work (lumo_ctx_set_timeout_drill)
  bool overlap = true;          // programmatic dependent launch between conv -> scan -> commit
  // Kind of the previous call that launched on this context.  Kernels that read some of their inputs
  // ahead of their dependency wait (commit: path and state; scan without convolution: state) get the
  // overlap attribute only when the call before them cannot have written those inputs.
  enum Call { kNone = 0, kVerify, kCommit, kCommitVerify, kOther };
  int last_call = kNone;
  bool timing = false;
  std::vector<cudaEvent_t> ev_start, ev_stop;
  std::vector<int> ev_kind;
};

struct lumo_tree_desc {
  lumo_ctx* ctx = nullptr;
  int B = 0, N = 0, Ns = 0;
  std::vector<lumo::HostTree> trees;     // per sequence
  // device tables (one allocation), all int32
  int32_t* dev = nullptr;
  int32_t* d_parent = nullptr;    // [B, N]
  int32_t* d_depth = nullptr;     // [B, N]
  int32_t* d_slot = nullptr;      // [B, N]
  int32_t* d_slot_inv = nullptr;  // [B, Ns]
  int32_t* d_win = nullptr;       // [B, Ns, 4] per entry of the conv visiting order: source rows (physical), -1/-2/-3 = history rows, INT32_MIN = padding row
  int32_t* d_child_off = nullptr; // [B, N+2]
  int32_t* d_child_list = nullptr;// [B, N]
  int32_t* d_conv_prog = nullptr; // [B, Ns] conv visiting order (depth first): physical row | flag << 16; flag 0 = fetch the whole
                                  // window, 1 = previous row is the parent (window slides), 2 = same parent as the previous row
                                  // (only the own row changes), 3 = padding row (zeros)
  int32_t* d_sched[2] = {nullptr, nullptr};   // [B, max_ops]  lean / full (every node's state materialised)
  int32_t* d_nops[2] = {nullptr, nullptr};    // [B]
  int max_ops[2] = {0, 0};
  int max_levels[2] = {0, 0};     // stack levels the schedule needs
  int max_depth = 0;              // deepest node over the batch
  // Gram-form scan tables (present when max_depth <= 16): the trees are cut into groups of at most
  // 64 nodes (prefix path + complete subtrees); G = number of groups over the batch
  int n_groups = 0;
  int max_group_nodes = 0;        // largest group (the scan picks a 32-node tile when every group fits it)
  int32_t* d_tc_group = nullptr;  // [G, 4]  sequence b, node count, first-group-of-b flag, 0
  int32_t* d_tc_meta = nullptr;   // [G, 64] physical row | depth << 16 | emit << 24 of the node at position pi
  uint8_t* d_tc_anc = nullptr;    // [G, 64, 16] positions of the ancestors, root first, then the node's own position
  uint8_t* d_tc_lvl = nullptr;    // [G, 20] lvl[d] = number of group nodes of depth <= d (lvl[0] = 0)
  // Which tail the Gram-form scan takes by default.  The level-by-level substitution costs one round per
  // eight nodes of a level, the closed-form tail a fixed part plus a part per node: thin, deep trees (a
  // spine with small side branches) are cheaper in closed form, wide ones by levels.
  bool closed_form_pays = false;
  // the same comparison for the closed form whose output sum is one tensor-core product (0.3 + 0.078 per node):
  // it pays on more trees, but only in launches of several waves, where an item's instruction count rather than
  // its latency sets the pace
  bool tensor_tail_pays = false;
  uint32_t* d_vis = nullptr;      // [B, N, 8] attention visibility over physical slots (present when Ns <= 256)
  uint32_t* d_slot_used = nullptr;// [B, 8] slots that hold a node
};

namespace lumo {

// ---- kernel-side views -----------------------------------------------------------------
struct LayerPtrs {
  void* q; void* k; void* v;
  const void* alpha; const void* beta;
  const float* a_log; const float* dt_bias;
  const void* x; const void* conv_w; const void* conv_b; void* conv_hist;
  float* state; const int32_t* state_row;
  void* out;
  const int32_t* snap_nodes; float* snap_out;
  int32_t* status;
};

struct LayerBatch {
  LayerPtrs l[kMaxLayers];
};

struct Shape {
  int B, N, Ns, Hk, Hv, d, C;
  int in_dtype, gate_dtype, out_dtype;
  float scale; int l2norm; float l2_eps;
  int n_state_rows;
  int snapshot_mode, n_snap;
  int n_layers;
  int gate_mode;
  int debug_skip_mma;   // test aid of the tensor-core scan: issue no tensor-core work, let the bounded wait run out
};

// What the fused commit + verify scan needs of the previous cycle: its layers (recorded k, v, gates,
// status), its tree (parent, slot) and the device-resident accepted path.
constexpr int kFusedMaxPath = 16;
struct FusedPrev {
  LayerBatch lb;
  const int32_t* parent; const int32_t* slot; int N, Ns;
  const int32_t* accepted; const int32_t* len; int lmax;
  int hist_in_kernels;   // 1: the conv reads the committed history through the path and the scan writes it back
};

struct TreeDev {
  const int32_t* parent; const int32_t* depth; const int32_t* slot; const int32_t* slot_inv;
  const int32_t* win; const int32_t* conv_prog; const int32_t* sched; const int32_t* nops; int max_ops; int max_levels;
  const int32_t* child_off; const int32_t* child_list;   // [B, N+2] CSR (entry 0 = pre-tree state), [B, N]
  const int32_t* tc_group; const int32_t* tc_meta; const uint8_t* tc_anc; const uint8_t* tc_lvl; int n_groups; int max_group_nodes;
};

void build_gram_groups(const int32_t* parent, int N, const HostTree& t, std::vector<GramGroup>* out);
// host-side tree tables (tree_desc.cpp)
bool build_tree(const int32_t* parent, const int32_t* slot, int N, int Ns, HostTree* t,
                int* levels_lean, int* levels_full, std::string* err);

// Programmatic dependent launch (sm_90+): a kernel launched with the attribute may start while its
// predecessor in the stream is still running; it must call pdl_wait() before touching anything the
// predecessor writes (or writing anything the predecessor reads), and the predecessor lets it in with
// pdl_trigger().  Rule used here: a kernel triggers only AFTER its own wait, so that everything older
// than its predecessor has completed by the time its dependent starts.
#ifdef __CUDACC__
// Gates of one (physical row, value head) as the recurrence consumes them: the stored values, or in
// raw-gate mode alpha = exp(-exp(a_log) softplus(g + dt_bias)), beta = sigmoid(b), in fp32.  Every
// kernel goes through this one function, so verify and commit see bit-identical gates.
__device__ __forceinline__ float2 load_gates(const LayerPtrs& L, const Shape& s, size_t i, int hv) {
  float a, b;
  if (s.gate_dtype == LUMO_BF16) {
    a = __uint_as_float((uint32_t)reinterpret_cast<const unsigned short*>(L.alpha)[i] << 16);
    b = __uint_as_float((uint32_t)reinterpret_cast<const unsigned short*>(L.beta)[i] << 16);
  } else {
    a = reinterpret_cast<const float*>(L.alpha)[i];
    b = reinterpret_cast<const float*>(L.beta)[i];
  }
  if (s.gate_mode == 1) {
    const float x = a + L.dt_bias[hv];
    const float sp = x > 20.f ? x : log1pf(expf(x));
    a = expf(-expf(L.a_log[hv]) * sp);
    b = 1.f / (1.f + expf(-b));
  }
  return make_float2(a, b);
}

// Accepted-path check; every CTA of a sequence reaches the same answer.  Order of checks: length,
// then per entry range, root, link.  The path's entries and their parents were staged in shared memory
// (parent -2 marks an entry outside [0, N)).
__device__ __forceinline__ int check_path_staged(const int* acc, const int* par, int N, int len, int lmax) {
  if (len < 0 || len > lmax) return LUMO_SEQ_BAD_LEN;
  int prev = -1;
  for (int t = 0; t < len; ++t) {       // bounded by lmax
    const int a = acc[t];
    if (a < 0 || a >= N) return LUMO_SEQ_BAD_NODE;
    if (t == 0) { if (par[t] != -1) return LUMO_SEQ_BAD_ROOT; }
    else if (par[t] != prev) return LUMO_SEQ_BAD_LINK;
    prev = a;
  }
  return LUMO_SEQ_OK;
}

// attention-side sequence check: the cache row exists and context plus suffix fit the row
__device__ __forceinline__ int seq_check(int ctx, int crow, int Ns, int n_rows, int max_pos) {
  if (crow < 0 || crow >= n_rows) return LUMO_SEQ_BAD_ROW;
  if (ctx < 0 || ctx > max_pos - Ns) return LUMO_SEQ_BAD_CTX;
  return LUMO_SEQ_OK;
}

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

// Largest thread-block cluster (16, 8, 4, 2 or 1 CTAs of `threads` threads along x) that the current
// device schedules for `kern`; 16 needs the non-portable opt-in.  Looked up once per device and kernel
// (`cache` is the caller's static table, zero-initialised).
template <typename K>
int max_cluster_ctas(K kern, int threads, int (&cache)[64]) {
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return 1;
  if (cache[dev] == 0) {
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.blockDim = dim3(threads);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    int c = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess ? 16 : 8;
    for (; c > 1; c >>= 1) {                               // bounded: at most four sizes
      int fit = 0;
      cfg.gridDim = dim3(c, 1);
      attr[0].val.clusterDim.x = c;
      if (cudaOccupancyMaxActiveClusters(&fit, kern, &cfg) == cudaSuccess && fit > 0) break;
    }
    (void)cudaGetLastError();
    cache[dev] = c;
  }
  return cache[dev];
}

// launch of a kernel whose CTAs form clusters of `cluster` along x
template <typename... KArgs, typename... Args>
cudaError_t launch_cluster_kernel(void (*kern)(KArgs...), dim3 grid, dim3 block, int cluster, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

template <typename... KArgs, typename... Args>
cudaError_t launch_kernel(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                          Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
#endif

// launchers (kernels.cu); all return cudaError_t and only enqueue
cudaError_t launch_conv(const Shape& s, const TreeDev& t, const LayerBatch& lb, bool pdl, cudaStream_t st);
// entries of the visiting order one CTA of the convolution takes (16, 8 or 4: fewer when the grid would not cover the GPU)
int conv_rows_per_cta(int C, int Ns, int seqs, int sms);
// same convolution reading the history the previous cycle's accepted path would commit (not yet in memory)
cudaError_t launch_conv_fused(const Shape& s, const TreeDev& t, const LayerBatch& lb, const FusedPrev& fp, bool pdl,
                              cudaStream_t st);
cudaError_t launch_scan(const Shape& s, const TreeDev& t, const LayerBatch& lb, float* stack,
                        int grid, cudaStream_t st);
// persistent grid size (CTAs resident at once) and the stack scratch it needs
cudaError_t scan_plan(const Shape& s, const TreeDev& t, int sm_count, int* grid, size_t* stack_bytes);
// acceptance walk (accept.cu)
struct AcceptView {
  int V, mode;
  const int32_t* token; const float* p_target; const float* q_draft; const float* uniforms; const float* noise;
  float* work;
};
cudaError_t launch_accept(const TreeDev& t, int B, int N, int Ns, const AcceptView& a, int lmax, int32_t* accepted,
                          int32_t* len, int32_t* next_token, int32_t* final_node, cudaStream_t st);
// fused draft selection (select.cu)
cudaError_t launch_select(const void* logits, int dtype, int rows, int V, int split, int32_t* spine, int32_t* cand,
                          cudaStream_t st);
// Gram-form scan on tcgen05 (scan_gram.cu)
bool gram_supported(const Shape& s, int max_depth);
// tail: 0 level-by-level substitution, 1 closed form (per-node back substitution, one output pass over the path),
// 2 closed form with the output sum as one tensor-core product
cudaError_t launch_scan_gram(const Shape& s, const TreeDev& t, const LayerBatch& lb, int sm_count, bool pdl, int tail,
                             cudaStream_t st);
// same scan, first replaying the previous cycle's accepted path into the state it has just loaded
cudaError_t launch_scan_gram_fused(const Shape& s, const TreeDev& t, const LayerBatch& lb, const FusedPrev& fp,
                                   int sm_count, bool pdl, int tail, cudaStream_t st);
// solved Gram form on tcgen05 (scan_solve.cu): the triangular system solved on scalars, one state product
cudaError_t launch_scan_solve(const Shape& s, const TreeDev& t, const LayerBatch& lb, int sm_count, bool pdl,
                              cudaStream_t st);
cudaError_t launch_scan_solve_fused(const Shape& s, const TreeDev& t, const LayerBatch& lb, const FusedPrev& fp,
                                    int sm_count, bool pdl, cudaStream_t st);
// device address of the built-in stack on `device` (which must be current); looked up once per device
cudaError_t static_stack_address(int device, float** ptr);
cudaError_t launch_commit(const Shape& s, const TreeDev& t, const LayerBatch& lb, const int32_t* accepted,
                          const int32_t* len, int lmax, bool with_state, bool with_hist, bool pdl, cudaStream_t st);
cudaError_t launch_path_from_node(const TreeDev& t, int B, int N, const int32_t* node, int lmax,
                                  int32_t* accepted, int32_t* len, int32_t* status, cudaStream_t st);

// ---- attention half (attn.cu) ------------------------------------------------------------
struct AttnShape {
  int B, N, Ns, Hq, Hkv, S, n_rows, max_pos, layout;
  float scale;
  const int32_t* ctx_len; const int32_t* cache_row;
};
struct AttnLayerPtrs {
  void* k_cache; void* v_cache; const void* q; float* out; float* lse; int32_t* status;
};
struct AttnArgs {
  const void* q;
  float* out; float* lse;
  float* part_o; float* part_lse;
  int2* unit_slots;   // per unit: first slot and slot count of its segments, written by the attention kernel
  uint32_t* fail_flag;   // set to launch_id by an attention CTA whose bounded wait ran out
  uint32_t launch_id;    // distinct per launch (never 0), so that the flag needs no clearing
  const int32_t* ctx_len; const int32_t* cache_row;
  const uint32_t* vis; const uint32_t* used;
  int32_t* status;
  int B, N, Ns, Hq, Hkv, G, RT, n_rows, max_pos;
  int S;   // partitions per unit; 0: the CTAs share the tile list evenly
  int C;   // CTAs of the attention launch
  int layout;   // 0: cache [row, position, head, dh]; 1: [row, head, position, dh]
  float scale_log2;
};
// one attention launch: the tensor maps of the layer's two caches, the kernel arguments and the grid
struct AttnPlan {
  CUtensorMap tk, tv;
  AttnArgs a;
  dim3 grid;
};
struct KvLayers {
  void* k[kMaxAttnLayers]; void* v[kMaxAttnLayers];
  const void* kn[kMaxAttnLayers]; const void* vn[kMaxAttnLayers];
  int32_t* status[kMaxAttnLayers];
};
struct KvShape {
  int B, N, Ns, Hkv, n_rows, max_pos, layout;
  const int32_t* ctx_len; const int32_t* cache_row;
  const int32_t* parent; const int32_t* slot;
};

int attn_row_tiles(int G, int N);
// scratch for the segments' partial results
size_t attn_scratch_bytes(const AttnShape& s, int sm_count);
cudaError_t attn_plan(const AttnShape& s, const AttnLayerPtrs& p, const uint32_t* vis, const uint32_t* used, float* scratch,
                      int sm_count, uint32_t launch_id, AttnPlan* plan, std::string* err);
cudaError_t launch_attn(const AttnPlan& plan, cudaStream_t st);
cudaError_t launch_attn_merge(const AttnPlan& plan, cudaStream_t st);
cudaError_t launch_kv_write(const KvLayers& L, const KvShape& s, int n_layers, cudaStream_t st);
cudaError_t launch_kv_publish(const KvLayers& L, const KvShape& s, int n_layers, const int32_t* accepted, const int32_t* len,
                              int lmax, int32_t* ctx_len_out, cudaStream_t st);

}  // namespace lumo
