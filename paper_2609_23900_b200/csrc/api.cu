// extern "C" entry points of liblumo_gdn: argument checking and launch orchestration.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <new>

#include "internal.h"

using namespace lumo;

namespace {

thread_local std::string g_create_err;

int fail(lumo_ctx* ctx, int code, const std::string& msg) {
  if (ctx) ctx->err = msg; else g_create_err = msg;
  return code;
}

int cuda_fail(lumo_ctx* ctx, cudaError_t e, const char* what) {
  return fail(ctx, LUMO_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

// Checks the layer array and fills the kernel-side views.  `need_out`: verify needs out.
int prepare(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_gdn_args* layers, int n_layers,
            bool for_verify, Shape* s, LayerBatch* lb) {
  if (!ctx || !desc || !layers) return fail(ctx, LUMO_ERR_ARG, "null ctx, desc or layers");
  if (desc->ctx != ctx) return fail(ctx, LUMO_ERR_ARG, "descriptor belongs to another context");
  if (ctx->device < 0) return fail(ctx, LUMO_ERR_UNSUPPORTED, "host-only context cannot launch");
  if (n_layers < 1 || n_layers > kMaxLayers)
    return fail(ctx, LUMO_ERR_ARG, "n_layers must be in [1, " + std::to_string(kMaxLayers) + "]");
  const lumo_gdn_args& a0 = layers[0];
  if (a0.d != 64 && a0.d != 128) return fail(ctx, LUMO_ERR_UNSUPPORTED, "d must be 64 or 128");
  if (a0.Hk < 1 || a0.Hv < 1 || a0.Hv % a0.Hk != 0)
    return fail(ctx, LUMO_ERR_UNSUPPORTED, "Hv must be a positive multiple of Hk");
  for (int dt : {a0.in_dtype, a0.gate_dtype, a0.out_dtype})
    if (dt != LUMO_F32 && dt != LUMO_BF16) return fail(ctx, LUMO_ERR_UNSUPPORTED, "dtype must be f32 or bf16");
  if (a0.snapshot_mode < 0 || a0.snapshot_mode > 2) return fail(ctx, LUMO_ERR_ARG, "snapshot_mode must be 0, 1 or 2");
  if (a0.n_state_rows < 1) return fail(ctx, LUMO_ERR_ARG, "n_state_rows must be positive");
  if (a0.gate_mode != 0 && a0.gate_mode != 1) return fail(ctx, LUMO_ERR_ARG, "gate_mode must be 0 or 1");
  std::memset(s, 0, sizeof(*s));
  s->B = desc->B; s->N = desc->N; s->Ns = desc->Ns;
  s->Hk = a0.Hk; s->Hv = a0.Hv; s->d = a0.d; s->C = 2 * a0.Hk * a0.d + a0.Hv * a0.d;
  s->in_dtype = a0.in_dtype; s->gate_dtype = a0.gate_dtype; s->out_dtype = a0.out_dtype;
  s->scale = a0.scale; s->l2norm = a0.qk_l2norm; s->l2_eps = a0.l2_eps;
  s->n_state_rows = a0.n_state_rows;
  s->snapshot_mode = for_verify ? a0.snapshot_mode : 0;
  s->n_snap = a0.snapshot_mode == 2 ? desc->N : a0.n_snap;
  s->n_layers = n_layers;
  s->gate_mode = a0.gate_mode;
  s->debug_skip_mma = ctx->timeout_drill ? 1 : 0;
  if (for_verify && a0.snapshot_mode == 1 && (a0.n_snap < 1 || a0.n_snap > kMaxNodes))
    return fail(ctx, LUMO_ERR_ARG, "n_snap must be in [1, 256] in snapshot list mode");
  for (int l = 0; l < n_layers; ++l) {
    const lumo_gdn_args& a = layers[l];
    const std::string at = " (layer " + std::to_string(l) + ")";
    if (a.Hk != a0.Hk || a.Hv != a0.Hv || a.d != a0.d || a.in_dtype != a0.in_dtype ||
        a.gate_dtype != a0.gate_dtype || a.out_dtype != a0.out_dtype || a.scale != a0.scale ||
        a.qk_l2norm != a0.qk_l2norm || a.l2_eps != a0.l2_eps || a.n_state_rows != a0.n_state_rows ||
        a.snapshot_mode != a0.snapshot_mode || a.n_snap != a0.n_snap || (a.x == nullptr) != (a0.x == nullptr) ||
        a.gate_mode != a0.gate_mode)
      return fail(ctx, LUMO_ERR_ARG, "all layers must share shape, dtypes and options" + at);
    if (!a.q || !a.k || !a.v || !a.alpha || !a.beta || !a.state || !a.state_row)
      return fail(ctx, LUMO_ERR_ARG, "q, k, v, alpha, beta, state and state_row are required" + at);
    if (a.gate_mode == 1 && (!a.a_log || !a.dt_bias))
      return fail(ctx, LUMO_ERR_ARG, "raw gates need a_log and dt_bias" + at);
    if (for_verify && !a.out) return fail(ctx, LUMO_ERR_ARG, "out is required" + at);
    if (a.x && (!a.conv_w || !a.conv_hist))
      return fail(ctx, LUMO_ERR_ARG, "x needs conv_w and conv_hist" + at);
    if (for_verify && a.snapshot_mode != 0 && !a.snap_out) return fail(ctx, LUMO_ERR_ARG, "snap_out is required" + at);
    if (for_verify && a.snapshot_mode == 1 && !a.snap_nodes) return fail(ctx, LUMO_ERR_ARG, "snap_nodes is required" + at);
    for (const void* p : {(const void*)a.q, (const void*)a.k, (const void*)a.v, a.x, a.conv_w, a.conv_b,
                          (const void*)a.conv_hist, (const void*)a.state, (const void*)a.out,
                          (const void*)a.snap_out})
      if (p && !aligned16(p)) return fail(ctx, LUMO_ERR_ARG, "tensor pointers must be 16-byte aligned" + at);
    LayerPtrs& p = lb->l[l];
    p.q = a.q; p.k = a.k; p.v = a.v; p.alpha = a.alpha; p.beta = a.beta;
    p.a_log = a.a_log; p.dt_bias = a.dt_bias;
    p.x = a.x; p.conv_w = a.conv_w; p.conv_b = a.conv_b; p.conv_hist = a.conv_hist;
    p.state = a.state; p.state_row = a.state_row; p.out = a.out;
    p.snap_nodes = a.snap_nodes; p.snap_out = a.snap_out; p.status = a.status;
  }
  return LUMO_OK;
}

constexpr size_t kTimingPool = 16384;

// Brackets one launch with events when timing is on.
template <typename F>
cudaError_t timed(lumo_ctx* ctx, int kind, cudaStream_t st, F launch) {
  const bool on = ctx->timing && ctx->ev_kind.size() < kTimingPool;
  size_t i = ctx->ev_kind.size();
  if (on) {
    cudaError_t e = cudaEventRecord(ctx->ev_start[i], st);
    if (e != cudaSuccess) return e;
  }
  cudaError_t e = launch();
  if (on && e == cudaSuccess) {
    e = cudaEventRecord(ctx->ev_stop[i], st);
    if (e == cudaSuccess) ctx->ev_kind.push_back(kind);
  }
  return e;
}

// Overlapping a kernel with its predecessor pays when both are a single wave of CTAs (the set-up and
// dependent-load chains hide under the predecessor's tail); with many waves it measured slower (the
// early CTAs only take slots from the predecessor), so it is limited to small launches.
bool use_overlap(const lumo_ctx* ctx, const Shape& s) {
  return ctx->overlap && (long long)s.n_layers * s.B * s.Hv <= 4LL * ctx->sm_count;
}

TreeDev tree_view(const lumo_tree_desc* d, int which) {
  TreeDev t;
  t.parent = d->d_parent; t.depth = d->d_depth; t.slot = d->d_slot; t.slot_inv = d->d_slot_inv;
  t.child_off = d->d_child_off; t.child_list = d->d_child_list;
  t.win = d->d_win; t.conv_prog = d->d_conv_prog; t.sched = d->d_sched[which]; t.nops = d->d_nops[which];
  t.max_ops = d->max_ops[which]; t.max_levels = d->max_levels[which];
  t.tc_group = d->d_tc_group; t.tc_meta = d->d_tc_meta; t.tc_anc = d->d_tc_anc; t.tc_lvl = d->d_tc_lvl;
  t.n_groups = d->n_groups;
  t.max_group_nodes = d->max_group_nodes;
  return t;
}

}  // namespace

extern "C" {

int lumo_ctx_create(int device, lumo_ctx** out) {
  if (!out) return fail(nullptr, LUMO_ERR_ARG, "out is null");
  *out = nullptr;
  if (device == -1) {   // host-only context: descriptors and their integer tables, no launches
    lumo_ctx* c = new (std::nothrow) lumo_ctx();
    if (!c) return fail(nullptr, LUMO_ERR_NOMEM, "out of host memory");
    c->device = -1;
    *out = c;
    return LUMO_OK;
  }
  int count = 0;
  cudaError_t e = cudaGetDeviceCount(&count);
  if (e != cudaSuccess) return cuda_fail(nullptr, e, "cudaGetDeviceCount");
  if (device < 0 || device >= count) return fail(nullptr, LUMO_ERR_ARG, "no such CUDA device");
  cudaDeviceProp prop;
  e = cudaGetDeviceProperties(&prop, device);
  if (e != cudaSuccess) return cuda_fail(nullptr, e, "cudaGetDeviceProperties");
  if (prop.major != 10)
    return fail(nullptr, LUMO_ERR_UNSUPPORTED, "this library holds sm_100a code only; device is sm_" +
                                                   std::to_string(prop.major) + std::to_string(prop.minor));
  lumo_ctx* c = new (std::nothrow) lumo_ctx();
  if (!c) return fail(nullptr, LUMO_ERR_NOMEM, "out of host memory");
  c->device = device;
  c->sm_count = prop.multiProcessorCount;
  *out = c;
  return LUMO_OK;
}

void lumo_ctx_destroy(lumo_ctx* ctx) {
  if (!ctx) return;
  if (ctx->device >= 0) {
    DeviceGuard g(ctx->device);
    if (ctx->scratch) cudaFree(ctx->scratch);
    if (ctx->attn_scratch) cudaFree(ctx->attn_scratch);
    for (cudaEvent_t e : ctx->ev_start) cudaEventDestroy(e);
    for (cudaEvent_t e : ctx->ev_stop) cudaEventDestroy(e);
  }
  delete ctx;
}

const char* lumo_last_error(const lumo_ctx* ctx) { return ctx ? ctx->err.c_str() : g_create_err.c_str(); }

int64_t lumo_ctx_scratch_bytes(const lumo_ctx* ctx) {
  return ctx ? (int64_t)(ctx->scratch_bytes + ctx->attn_scratch_bytes) : 0;
}

int lumo_ctx_set_scan_algo(lumo_ctx* ctx, int algo) {
  if (!ctx) return LUMO_ERR_ARG;
  if (algo < 0 || algo > 5)
    return fail(ctx, LUMO_ERR_ARG, "scan algo must be 0 (auto), 1 (rank-1), 2 (Gram form, forward substitution), 3 (solved Gram form), 4 (Gram form, closed-form tail) or 5 (closed-form tail, output sum on the tensor core)");
  ctx->scan_algo = algo;
  return LUMO_OK;
}

int lumo_ctx_set_timeout_drill(lumo_ctx* ctx, int on) {
  if (!ctx) return LUMO_ERR_ARG;
  ctx->timeout_drill = on != 0;
  return LUMO_OK;
}

int lumo_ctx_set_overlap(lumo_ctx* ctx, int on) {
  if (!ctx) return LUMO_ERR_ARG;
  ctx->overlap = on != 0;
  return LUMO_OK;
}

int lumo_ctx_timing_enable(lumo_ctx* ctx, int enable) {
  if (!ctx) return LUMO_ERR_ARG;
  if (ctx->device < 0) return fail(ctx, LUMO_ERR_UNSUPPORTED, "host-only context cannot launch");
  DeviceGuard g(ctx->device);
  if (enable && ctx->ev_start.empty()) {
    ctx->ev_start.resize(kTimingPool);
    ctx->ev_stop.resize(kTimingPool);
    for (size_t i = 0; i < kTimingPool; ++i) {
      cudaError_t e = cudaEventCreate(&ctx->ev_start[i]);
      if (e == cudaSuccess) e = cudaEventCreate(&ctx->ev_stop[i]);
      if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaEventCreate");
    }
    ctx->ev_kind.reserve(kTimingPool);
  }
  ctx->timing = enable != 0;
  return LUMO_OK;
}

int lumo_ctx_timing_read(lumo_ctx* ctx, int kind, int reset, int64_t* launches, double* total_ms) {
  if (!ctx || !launches || !total_ms || kind < 0 || kind >= LUMO_K_COUNT) return fail(ctx, LUMO_ERR_ARG, "bad argument");
  DeviceGuard g(ctx->device);
  *launches = 0;
  *total_ms = 0.0;
  for (size_t i = 0; i < ctx->ev_kind.size(); ++i) {
    if (ctx->ev_kind[i] != kind) continue;
    cudaError_t e = cudaEventSynchronize(ctx->ev_stop[i]);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, ctx->ev_start[i], ctx->ev_stop[i]);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "event read");
    *launches += 1;
    *total_ms += ms;
  }
  if (reset) ctx->ev_kind.clear();
  return LUMO_OK;
}

int lumo_tree_desc_create(lumo_ctx* ctx, int batch, int n_nodes, int n_slots, const int32_t* parent,
                          const int32_t* depth, const int32_t* slot, lumo_tree_desc** out) {
  if (!ctx || !out || !parent) return fail(ctx, LUMO_ERR_ARG, "null ctx, out or parent");
  *out = nullptr;
  if (batch < 1 || n_nodes < 1 || n_nodes > kMaxNodes || n_slots < n_nodes || n_slots > kMaxSlots)
    return fail(ctx, LUMO_ERR_ARG, "need batch >= 1, 1 <= n_nodes <= 256, n_nodes <= n_slots <= 1024");
  lumo_tree_desc* d = new (std::nothrow) lumo_tree_desc();
  if (!d) return fail(ctx, LUMO_ERR_NOMEM, "out of host memory");
  d->ctx = ctx; d->B = batch; d->N = n_nodes; d->Ns = n_slots;
  d->trees.resize(batch);
  const int B = batch, N = n_nodes, Ns = n_slots;
  for (int b = 0; b < B; ++b) {
    std::string err;
    int lv[2];
    if (!build_tree(parent + (size_t)b * N, slot ? slot + (size_t)b * N : nullptr, N, Ns, &d->trees[b],
                    &lv[0], &lv[1], &err)) {
      delete d;
      return fail(ctx, LUMO_ERR_TREE, "sequence " + std::to_string(b) + ": " + err);
    }
    if (depth)
      for (int i = 0; i < N; ++i)
        if (depth[(size_t)b * N + i] != d->trees[b].tab[LUMO_TAB_DEPTH][i]) {
          delete d;
          return fail(ctx, LUMO_ERR_TREE, "sequence " + std::to_string(b) + ": depth[" + std::to_string(i) +
                                              "] does not match the parent array");
        }
    for (int w = 0; w < 2; ++w) {
      d->max_levels[w] = std::max(d->max_levels[w], lv[w]);
      d->max_ops[w] = std::max(d->max_ops[w], (int)d->trees[b].tab[LUMO_TAB_SCHEDULE + w].size());
    }
  }
  // one device allocation holding every table
  std::vector<int32_t> h;
  auto reserve = [&](size_t n) { size_t off = h.size(); h.resize(off + ((n + 3) / 4) * 4, 0); return off; };
  const size_t o_parent = reserve((size_t)B * N), o_depth = reserve((size_t)B * N), o_slot = reserve((size_t)B * N);
  const size_t o_inv = reserve((size_t)B * Ns), o_win = reserve((size_t)B * Ns * 4);
  const size_t o_prog = reserve((size_t)B * Ns);
  const size_t o_winv = reserve((size_t)B * Ns * 4);
  const size_t o_coff = reserve((size_t)B * (N + 2)), o_clist = reserve((size_t)B * N);
  size_t o_sched[2], o_nops[2];
  for (int w = 0; w < 2; ++w) { o_sched[w] = reserve((size_t)B * d->max_ops[w]); o_nops[w] = reserve(B); }
  for (int b = 0; b < B; ++b)
    for (int i = 0; i < N; ++i) d->max_depth = std::max(d->max_depth, (int)d->trees[b].tab[LUMO_TAB_DEPTH][i]);
  const bool tc = d->max_depth <= 16;
  std::vector<std::vector<GramGroup>> groups(B);
  if (tc)
    for (int b = 0; b < B; ++b) {
      build_gram_groups(parent + (size_t)b * N, N, d->trees[b], &groups[b]);
      d->n_groups += (int)groups[b].size();
      auto& tab = d->trees[b].tab[LUMO_TAB_GRAM_GROUPS];
      tab.push_back((int32_t)groups[b].size());
      for (const GramGroup& gr : groups[b]) {
        d->max_group_nodes = std::max(d->max_group_nodes, (int)gr.nodes.size());
        tab.push_back((int32_t)gr.nodes.size());
        tab.insert(tab.end(), gr.nodes.begin(), gr.nodes.end());
        tab.insert(tab.end(), gr.emit.begin(), gr.emit.end());
      }
    }
  const size_t G = (size_t)d->n_groups;
  const size_t o_tc_group = tc ? reserve(G * 4) : 0, o_tc_meta = tc ? reserve(G * 64) : 0;
  const size_t o_tc_anc = tc ? reserve(G * 64 * 4) : 0, o_tc_lvl = tc ? reserve(G * 5) : 0;
  const bool attn = Ns <= kMaxAttnSlots;
  const size_t o_vis = attn ? reserve((size_t)B * N * 8) : 0, o_used = attn ? reserve((size_t)B * 8) : 0;
  size_t gi = 0;
  long long subst_rounds = 0, group_nodes = 0;     // over all groups: rounds of the substitution, nodes
  for (int b = 0; b < B; ++b) {
    const HostTree& t = d->trees[b];
    if (attn) {
      const int W = (Ns + 31) / 32;
      for (int i = 0; i < N; ++i)
        for (int w = 0; w < W; ++w) {
          const int32_t m = t.tab[LUMO_TAB_ATTN_VIS][(size_t)i * W + w];
          h[o_vis + ((size_t)b * N + i) * 8 + w] = m;
          h[o_used + (size_t)b * 8 + w] |= m;       // every node sees its own slot
        }
    }
    for (int i = 0; i < N; ++i) {
      h[o_parent + (size_t)b * N + i] = parent[(size_t)b * N + i];
      h[o_depth + (size_t)b * N + i] = t.tab[LUMO_TAB_DEPTH][i];
      h[o_slot + (size_t)b * N + i] = slot ? slot[(size_t)b * N + i] : i;
    }
    for (int sidx = 0; sidx < Ns; ++sidx) h[o_inv + (size_t)b * Ns + sidx] = t.tab[LUMO_TAB_SLOT_INV][sidx];
    // conv windows per PHYSICAL row, entries in physical rows (or -1..-3 = history rows);
    // a padding row holds INT32_MIN
    for (int sidx = 0; sidx < Ns; ++sidx) {
      const int node = t.tab[LUMO_TAB_SLOT_INV][sidx];
      for (int j = 0; j < 4; ++j) {
        int w = INT32_MIN;
        if (node >= 0) {
          w = t.tab[LUMO_TAB_ANC_WIN][node * 4 + j];
          if (w >= 0) w = h[o_slot + (size_t)b * N + w];
        }
        h[o_win + ((size_t)b * Ns + sidx) * 4 + j] = w;
      }
    }
    for (int i = 0; i < N + 2; ++i) h[o_coff + (size_t)b * (N + 2) + i] = t.tab[LUMO_TAB_CHILD_OFF][i];
    for (int i = 0; i < N; ++i) h[o_clist + (size_t)b * N + i] = t.tab[LUMO_TAB_CHILD_LIST][i];
    {
      // conv visiting order: depth-first preorder, so that most rows find three of their four taps
      // already in the registers of the thread that handled the previous row
      const auto& coff = t.tab[LUMO_TAB_CHILD_OFF];
      const auto& clist = t.tab[LUMO_TAB_CHILD_LIST];
      std::vector<int> stack, order;
      for (int c = coff[1] - 1; c >= coff[0]; --c) stack.push_back(clist[c]);
      while (!stack.empty()) {
        const int n = stack.back(); stack.pop_back();
        order.push_back(n);
        for (int c = coff[n + 2] - 1; c >= coff[n + 1]; --c) stack.push_back(clist[c]);
      }
      size_t k = 0;
      for (size_t pidx = 0; pidx < order.size(); ++pidx, ++k) {
        const int n = order[pidx];
        int flag = 0;
        if (pidx > 0) {
          const int prev = order[pidx - 1];
          const int pn = parent[(size_t)b * N + n], pp = parent[(size_t)b * N + prev];
          if (pn == prev) flag = 1;
          else if (pn == pp) flag = 2;
        }
        h[o_prog + (size_t)b * Ns + k] = h[o_slot + (size_t)b * N + n] | (flag << 16);
      }
      for (int sidx = 0; sidx < Ns; ++sidx)
        if (t.tab[LUMO_TAB_SLOT_INV][sidx] < 0) h[o_prog + (size_t)b * Ns + k++] = sidx | (3 << 16);
      // the windows in the same visiting order, so that the kernel fetches order and window together
      for (int e = 0; e < Ns; ++e) {
        const int sidx = h[o_prog + (size_t)b * Ns + e] & 0xFFFF;
        for (int j = 0; j < 4; ++j) h[o_winv + ((size_t)b * Ns + e) * 4 + j] = h[o_win + ((size_t)b * Ns + sidx) * 4 + j];
      }
    }
    for (int w = 0; w < 2; ++w) {
      const auto& ops = t.tab[LUMO_TAB_SCHEDULE + w];
      std::copy(ops.begin(), ops.end(), h.begin() + o_sched[w] + (size_t)b * d->max_ops[w]);
      h[o_nops[w] + b] = (int32_t)ops.size();
    }
    if (tc) {
      for (size_t k = 0; k < groups[b].size(); ++k, ++gi) {
        const GramGroup& gr = groups[b][k];
        const int n = (int)gr.nodes.size();
        h[o_tc_group + gi * 4 + 0] = b;
        h[o_tc_group + gi * 4 + 1] = n;
        h[o_tc_group + gi * 4 + 2] = k == 0;
        std::vector<int> pos(N, -1);
        for (int pi = 0; pi < n; ++pi) pos[gr.nodes[pi]] = pi;
        uint8_t* lvl = reinterpret_cast<uint8_t*>(h.data() + o_tc_lvl) + gi * 20;
        uint8_t* anc = reinterpret_cast<uint8_t*>(h.data() + o_tc_anc) + gi * 64 * 16;
        for (int pi = 0; pi < n; ++pi) {
          const int node = gr.nodes[pi];
          const int dep = t.tab[LUMO_TAB_DEPTH][node];
          h[o_tc_meta + gi * 64 + pi] = h[o_slot + (size_t)b * N + node] | (dep << 16) | ((int)gr.emit[pi] << 24);
          int cur = parent[(size_t)b * N + node];
          anc[pi * 16 + dep - 1] = (uint8_t)pi;
          for (int j = dep - 2; j >= 0; --j) { anc[pi * 16 + j] = (uint8_t)pos[cur]; cur = parent[(size_t)b * N + cur]; }
          for (int dd = dep; dd < 20; ++dd) lvl[dd] += 1;      // lvl[d] = members of depth <= d
        }
        for (int dd = 1; dd < 20; ++dd) subst_rounds += (lvl[dd] - lvl[dd - 1] + 7) / 8;
        group_nodes += n;
      }
    }
  }
  // measured on B200 (us per item): substitution 0.45 per round, closed form 1.7 + 0.08 per node; the
  // closed form is taken when it wins by a margin (28-node spine trees of depth 12: 18.5 -> 17.0 us per
  // launch at batch 8; 64-node trees of depth 8 stay with the substitution: 19.1 against 20.5 us)
  d->closed_form_pays = tc && 100 * subst_rounds > 600 * (long long)G + 18 * group_nodes;
  // measured with the tensor-core sum (launch times, us, substitution against it): 48 layers of 32-node trees
  // 190 -> 175, 256-node chains 225 -> 190, random 256-node trees 236 -> 218; a 255-child star 177 -> 200 and
  // single-wave launches (64-node trees at batch 8: equal within 1%, at four times the error) stay
  d->tensor_tail_pays = tc && 450 * subst_rounds > 300 * (long long)G + 78 * group_nodes;
  if (ctx->device < 0) { *out = d; return LUMO_OK; }   // host-only: tables stay on the host
  DeviceGuard g(ctx->device);
  cudaError_t e = cudaMalloc(&d->dev, h.size() * sizeof(int32_t));
  if (e != cudaSuccess) { delete d; return cuda_fail(ctx, e, "cudaMalloc(tree tables)"); }
  e = cudaMemcpy(d->dev, h.data(), h.size() * sizeof(int32_t), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) { cudaFree(d->dev); delete d; return cuda_fail(ctx, e, "cudaMemcpy(tree tables)"); }
  d->d_parent = d->dev + o_parent; d->d_depth = d->dev + o_depth; d->d_slot = d->dev + o_slot;
  d->d_slot_inv = d->dev + o_inv; d->d_win = d->dev + o_winv; d->d_conv_prog = d->dev + o_prog;
  d->d_child_off = d->dev + o_coff; d->d_child_list = d->dev + o_clist;
  for (int w = 0; w < 2; ++w) { d->d_sched[w] = d->dev + o_sched[w]; d->d_nops[w] = d->dev + o_nops[w]; }
  if (tc) {
    d->d_tc_group = d->dev + o_tc_group;
    d->d_tc_meta = d->dev + o_tc_meta;
    d->d_tc_anc = reinterpret_cast<uint8_t*>(d->dev + o_tc_anc);
    d->d_tc_lvl = reinterpret_cast<uint8_t*>(d->dev + o_tc_lvl);
  }
  if (attn) {
    d->d_vis = reinterpret_cast<uint32_t*>(d->dev + o_vis);
    d->d_slot_used = reinterpret_cast<uint32_t*>(d->dev + o_used);
  }
  *out = d;
  return LUMO_OK;
}

void lumo_tree_desc_destroy(lumo_tree_desc* desc) {
  if (!desc) return;
  if (desc->dev) {
    DeviceGuard g(desc->ctx->device);
    cudaFree(desc->dev);
  }
  delete desc;
}

int lumo_tree_desc_get(const lumo_tree_desc* desc, int which, int b, const int32_t** data, int64_t* count) {
  if (!desc || !data || !count || which < 0 || which >= LUMO_TAB_COUNT || b < 0 || b >= desc->B) return LUMO_ERR_ARG;
  const auto& v = desc->trees[b].tab[which];
  *data = v.data();
  *count = (int64_t)v.size();
  return LUMO_OK;
}

int lumo_tree_path_from_node(lumo_ctx* ctx, const lumo_tree_desc* desc, const int32_t* node_dev, int lmax,
                             int32_t* accepted_dev, int32_t* len_dev, int32_t* status_dev, void* stream) {
  if (!ctx || !desc || !node_dev || !accepted_dev || !len_dev) return fail(ctx, LUMO_ERR_ARG, "null argument");
  if (desc->ctx != ctx) return fail(ctx, LUMO_ERR_ARG, "descriptor belongs to another context");
  if (lmax < 1) return fail(ctx, LUMO_ERR_ARG, "lmax must be positive");
  if (ctx->device < 0) return fail(ctx, LUMO_ERR_UNSUPPORTED, "host-only context cannot launch");
  DeviceGuard g(ctx->device);
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = timed(ctx, LUMO_K_PATH, st, [&] {
    return launch_path_from_node(tree_view(desc, 0), desc->B, desc->N, node_dev, lmax, accepted_dev, len_dev,
                                 status_dev, st);
  });
  ctx->last_call = lumo_ctx::kOther;
  return e == cudaSuccess ? LUMO_OK : cuda_fail(ctx, e, "path_from_node launch");
}

int lumo_tree_accept(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_accept_args* a, int lmax,
                     int32_t* accepted_dev, int32_t* len_dev, int32_t* next_token_dev, int32_t* final_node_dev,
                     void* stream) {
  if (!ctx || !desc || !a || !accepted_dev || !len_dev || !next_token_dev || !final_node_dev)
    return fail(ctx, LUMO_ERR_ARG, "null argument");
  if (desc->ctx != ctx) return fail(ctx, LUMO_ERR_ARG, "descriptor belongs to another context");
  if (ctx->device < 0) return fail(ctx, LUMO_ERR_UNSUPPORTED, "host-only context cannot launch");
  if (a->V < 1) return fail(ctx, LUMO_ERR_ARG, "V must be positive");
  if (a->mode != 0 && a->mode != 1) return fail(ctx, LUMO_ERR_ARG, "mode must be 0 (greedy) or 1 (rejection sampling)");
  if (lmax < desc->max_depth) return fail(ctx, LUMO_ERR_ARG, "lmax must be at least the tree depth");
  if (!a->token || !a->p_target) return fail(ctx, LUMO_ERR_ARG, "token and p_target are required");
  if (a->mode == 1 && (!a->q_draft || !a->uniforms || !a->noise || !a->work))
    return fail(ctx, LUMO_ERR_ARG, "rejection sampling needs q_draft, uniforms, noise and work");
  DeviceGuard g(ctx->device);
  AcceptView v;
  v.V = a->V; v.mode = a->mode; v.token = a->token; v.p_target = a->p_target; v.q_draft = a->q_draft;
  v.uniforms = a->uniforms; v.noise = a->noise; v.work = a->work;
  cudaError_t e = launch_accept(tree_view(desc, 0), desc->B, desc->N, desc->Ns, v, lmax, accepted_dev, len_dev,
                                next_token_dev, final_node_dev, (cudaStream_t)stream);
  ctx->last_call = lumo_ctx::kOther;
  return e == cudaSuccess ? LUMO_OK : cuda_fail(ctx, e, "accept launch");
}

int lumo_select_spine_top3(lumo_ctx* ctx, const lumo_select_args* a, int32_t* spine_dev, int32_t* cand_dev,
                           void* stream) {
  if (!ctx || !a || !a->logits || !spine_dev || !cand_dev) return fail(ctx, LUMO_ERR_ARG, "null argument");
  if (ctx->device < 0) return fail(ctx, LUMO_ERR_UNSUPPORTED, "host-only context cannot launch");
  if (a->rows < 1 || a->V < 3) return fail(ctx, LUMO_ERR_ARG, "need rows >= 1 and V >= 3");
  if (a->rows > 65535) return fail(ctx, LUMO_ERR_ARG, "at most 65535 rows per call");
  if (a->dtype != LUMO_F32 && a->dtype != LUMO_BF16) return fail(ctx, LUMO_ERR_ARG, "logits must be f32 or bf16");
  const int sp = a->split;
  if (sp != 0 && sp != 1 && sp != 2 && sp != 4 && sp != 8 && sp != 16)
    return fail(ctx, LUMO_ERR_ARG, "split must be 0, 1, 2, 4, 8 or 16");
  DeviceGuard g(ctx->device);
  cudaError_t e = launch_select(a->logits, a->dtype, a->rows, a->V, sp, spine_dev, cand_dev, (cudaStream_t)stream);
  ctx->last_call = lumo_ctx::kOther;
  if (e == cudaErrorInvalidConfiguration) {
    (void)cudaGetLastError();
    return fail(ctx, LUMO_ERR_UNSUPPORTED, "this device does not schedule clusters of that size");
  }
  return e == cudaSuccess ? LUMO_OK : cuda_fail(ctx, e, "select launch");
}

// Which tail the Gram-form scan takes: 0 level-by-level substitution, 1 closed form, 2 closed form with the output
// sum on the tensor core.  Automatic: thin deep trees take 2 (equal to 1 there, measured); other trees take 2 when
// the descriptor says it pays and the launch has several waves of items; everything else takes 0.
static int scan_tail(const lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo::Shape& s) {
  if (ctx->scan_algo == 5) return 2;
  if (ctx->scan_algo == 4) return 1;
  if (ctx->scan_algo != 0) return 0;
  if (desc->closed_form_pays) return 2;
  const long long items = (long long)s.n_layers * desc->n_groups * s.Hv;
  return desc->tensor_tail_pays && items > 2LL * ctx->sm_count ? 2 : 0;
}

int lumo_gdn_tree_verify(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_gdn_args* layers, int n_layers,
                         void* stream) {
  Shape s;
  LayerBatch lb;
  std::memset(&lb, 0, sizeof(lb));
  int rc = prepare(ctx, desc, layers, n_layers, true, &s, &lb);
  if (rc != LUMO_OK) return rc;
  DeviceGuard g(ctx->device);
  cudaStream_t st = (cudaStream_t)stream;
  const TreeDev t = tree_view(desc, s.snapshot_mode != 0 ? 1 : 0);
  const bool gram_ok = desc->d_tc_meta != nullptr && gram_supported(s, desc->max_depth);
  if (ctx->scan_algo >= 2 && !gram_ok)
    return fail(ctx, LUMO_ERR_UNSUPPORTED, "the Gram-form scan needs d = 128, bf16 operands, depth <= 16, no snapshots");
  // The Gram-form scan requests the pre-tree state ahead of its dependency wait.  Behind a convolution
  // that is safe (the convolution waits first, so whatever wrote the state has completed); launched
  // directly behind a call that rewrote the state it takes plain stream order instead.
  const int prev_call = ctx->last_call;
  ctx->last_call = lumo_ctx::kVerify;
  if (gram_ok && ctx->scan_algo != 1) {
    cudaError_t e = cudaSuccess;
    if (layers[0].x) {
      e = timed(ctx, LUMO_K_CONV, st, [&] { return launch_conv(s, t, lb, use_overlap(ctx, s), st); });
      if (e != cudaSuccess) return cuda_fail(ctx, e, "conv launch");
    }
    const bool state_fresh = !layers[0].x && (prev_call == lumo_ctx::kCommit || prev_call == lumo_ctx::kCommitVerify);
    e = timed(ctx, LUMO_K_SCAN, st, [&] {
      const bool pdl = use_overlap(ctx, s) && !state_fresh;
      return ctx->scan_algo == 3 ? launch_scan_solve(s, t, lb, ctx->sm_count, pdl, st)
                                 : launch_scan_gram(s, t, lb, ctx->sm_count, pdl, scan_tail(ctx, desc, s), st);
    });
    return e == cudaSuccess ? LUMO_OK : cuda_fail(ctx, e, "Gram-form scan launch");
  }
  int grid = 0;
  size_t stack_bytes = 0;
  cudaError_t e = scan_plan(s, t, ctx->sm_count, &grid, &stack_bytes);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "scan_plan");
  if (stack_bytes > ctx->scratch_bytes) {
    // first call with this shape: grow the scratch (synchronises; later calls allocate nothing)
    if (ctx->scratch) {
      e = cudaDeviceSynchronize();
      if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaDeviceSynchronize");
      cudaFree(ctx->scratch);
      ctx->scratch = nullptr;
      ctx->scratch_bytes = 0;
    }
    e = cudaMalloc(&ctx->scratch, stack_bytes);
    if (e != cudaSuccess) return fail(ctx, LUMO_ERR_NOMEM, std::string("scratch allocation failed: ") + cudaGetErrorString(e));
    ctx->scratch_bytes = stack_bytes;
  }
  if (layers[0].x) {
    e = timed(ctx, LUMO_K_CONV, st, [&] { return launch_conv(s, t, lb, use_overlap(ctx, s), st); });
    if (e != cudaSuccess) return cuda_fail(ctx, e, "conv launch");
  }
  e = timed(ctx, LUMO_K_SCAN, st, [&] {
    return launch_scan(s, t, lb, reinterpret_cast<float*>(ctx->scratch), grid, st);
  });
  return e == cudaSuccess ? LUMO_OK : cuda_fail(ctx, e, "scan launch");
}

int64_t lumo_static_stack_bytes(void) { return (int64_t)kStaticStackBytes; }

int lumo_conv_rows_per_cta(const lumo_ctx* ctx, const lumo_tree_desc* desc, int Hk, int Hv, int d, int n_layers) {
  if (!ctx || !desc || ctx->device < 0 || Hk < 1 || Hv < 1 || d < 1 || n_layers < 1) return 0;
  return conv_rows_per_cta(2 * Hk * d + Hv * d, desc->Ns, desc->B * n_layers, ctx->sm_count);
}

int lumo_gdn_tree_scan_static(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_gdn_args* layers,
                              int n_layers, void* stream) {
  Shape s;
  LayerBatch lb;
  std::memset(&lb, 0, sizeof(lb));
  int rc = prepare(ctx, desc, layers, n_layers, true, &s, &lb);
  if (rc != LUMO_OK) return rc;
  DeviceGuard g(ctx->device);
  cudaStream_t st = (cudaStream_t)stream;
  const TreeDev t = tree_view(desc, s.snapshot_mode != 0 ? 1 : 0);
  int grid = 0;
  size_t stack_bytes = 0;
  cudaError_t e = scan_plan(s, t, ctx->sm_count, &grid, &stack_bytes);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "scan_plan");
  if (stack_bytes > kStaticStackBytes)
    return fail(ctx, LUMO_ERR_UNSUPPORTED,
                "this shape needs " + std::to_string(stack_bytes) + " bytes of scan stack; the built-in stack holds " +
                    std::to_string(kStaticStackBytes) + " (use lumo_gdn_tree_verify, which allocates)");
  float* stack = nullptr;
  e = static_stack_address(ctx->device, &stack);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaGetSymbolAddress(built-in scan stack)");
  e = timed(ctx, LUMO_K_SCAN, st, [&] { return launch_scan(s, t, lb, stack, grid, st); });
  ctx->last_call = lumo_ctx::kVerify;
  return e == cudaSuccess ? LUMO_OK : cuda_fail(ctx, e, "scan launch");
}

int lumo_gdn_commit(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_gdn_args* layers, int n_layers,
                    const int32_t* accepted_dev, const int32_t* len_dev, int lmax, void* stream) {
  // the kernel stages the whole path in arrays of kMaxNodes entries: refused here, before anything else
  if (ctx && (lmax < 1 || lmax > kMaxNodes))
    return fail(ctx, LUMO_ERR_ARG, "lmax must be in [1, " + std::to_string(kMaxNodes) + "] (a path holds each node at most once)");
  Shape s;
  LayerBatch lb;
  std::memset(&lb, 0, sizeof(lb));
  int rc = prepare(ctx, desc, layers, n_layers, false, &s, &lb);
  if (rc != LUMO_OK) return rc;
  if (!accepted_dev || !len_dev) return fail(ctx, LUMO_ERR_ARG, "accepted_dev and len_dev are required");
  DeviceGuard g(ctx->device);
  cudaStream_t st = (cudaStream_t)stream;
  const TreeDev t = tree_view(desc, 0);
  // the commit reads the path, the operands and the state ahead of its dependency wait: overlap only
  // right behind a verify call (see commit_kernel)
  const bool pdl = use_overlap(ctx, s) && ctx->last_call == lumo_ctx::kVerify;
  ctx->last_call = lumo_ctx::kCommit;
  cudaError_t e = timed(ctx, LUMO_K_COMMIT, st, [&] {
    return launch_commit(s, t, lb, accepted_dev, len_dev, lmax, true, layers[0].x != nullptr, pdl, st);
  });
  return e == cudaSuccess ? LUMO_OK : cuda_fail(ctx, e, "commit launch");
}

int lumo_gdn_commit_verify(lumo_ctx* ctx, const lumo_tree_desc* prev_desc, const lumo_gdn_args* prev_layers,
                           const int32_t* accepted_dev, const int32_t* len_dev, int lmax,
                           const lumo_tree_desc* desc, const lumo_gdn_args* layers, int n_layers, void* stream) {
  if (ctx && (lmax < 1 || lmax > kMaxNodes))
    return fail(ctx, LUMO_ERR_ARG, "lmax must be in [1, " + std::to_string(kMaxNodes) + "] (a path holds each node at most once)");
  Shape ps, s;
  LayerBatch lb;
  FusedPrev fp;
  std::memset(&lb, 0, sizeof(lb));
  std::memset(&fp, 0, sizeof(fp));
  int rc = prepare(ctx, prev_desc, prev_layers, n_layers, false, &ps, &fp.lb);
  if (rc != LUMO_OK) return rc;
  rc = prepare(ctx, desc, layers, n_layers, true, &s, &lb);
  if (rc != LUMO_OK) return rc;
  if (!accepted_dev || !len_dev) return fail(ctx, LUMO_ERR_ARG, "accepted_dev and len_dev are required");
  if (prev_desc->B != desc->B) return fail(ctx, LUMO_ERR_ARG, "both trees must cover the same batch");
  if (ps.Hk != s.Hk || ps.Hv != s.Hv || ps.d != s.d || ps.in_dtype != s.in_dtype || ps.gate_dtype != s.gate_dtype ||
      ps.l2norm != s.l2norm || ps.l2_eps != s.l2_eps || ps.gate_mode != s.gate_mode || ps.n_state_rows != s.n_state_rows)
    return fail(ctx, LUMO_ERR_ARG, "both cycles must share shapes, dtypes and options");
  for (int l = 0; l < n_layers; ++l) {
    const lumo_gdn_args &p = prev_layers[l], &c = layers[l];
    if (p.state != c.state || p.state_row != c.state_row || p.conv_hist != c.conv_hist)
      return fail(ctx, LUMO_ERR_ARG, "both cycles must name the same state, state_row and conv_hist");
    if (p.k == c.k || p.v == c.v || (p.x && p.x == c.x))
      return fail(ctx, LUMO_ERR_ARG, "the previous cycle's operands must live in their own buffers");
    if (p.gate_mode == 1 && (p.a_log != c.a_log || p.dt_bias != c.dt_bias))
      return fail(ctx, LUMO_ERR_ARG, "both cycles must share a_log and dt_bias");
  }
  const bool gram_ok = desc->d_tc_meta != nullptr && gram_supported(s, desc->max_depth);
  const bool fused = gram_ok && ctx->scan_algo != 1 && desc->n_groups == desc->B && lmax <= kFusedMaxPath;
  if (!fused) {   // same result from the two separate calls
    rc = lumo_gdn_commit(ctx, prev_desc, prev_layers, n_layers, accepted_dev, len_dev, lmax, stream);
    if (rc != LUMO_OK) return rc;
    return lumo_gdn_tree_verify(ctx, desc, layers, n_layers, stream);
  }
  DeviceGuard g(ctx->device);
  cudaStream_t st = (cudaStream_t)stream;
  // The convolution waits on its predecessor before it reads anything, so it may always overlap, and
  // so may a scan launched behind it.  A fused scan (or the history launch) directly behind another
  // call reads the path and the state ahead of its dependency wait: overlap then only behind a verify.
  const bool pdl_conv = use_overlap(ctx, s);
  const bool pdl = pdl_conv && ctx->last_call == lumo_ctx::kVerify;
  const bool pdl_scan = pdl_conv && (layers[0].x != nullptr || ctx->last_call == lumo_ctx::kVerify);
  ctx->last_call = lumo_ctx::kCommitVerify;
  const TreeDev pt = tree_view(prev_desc, 0);
  const TreeDev t = tree_view(desc, 0);
  fp.parent = pt.parent; fp.slot = pt.slot; fp.N = prev_desc->N; fp.Ns = prev_desc->Ns;
  fp.accepted = accepted_dev; fp.len = len_dev; fp.lmax = lmax;
  cudaError_t e = cudaSuccess;
  // Convolution history of the accepted path.  With a convolution in this cycle the two kernels take
  // care of it (the conv reads the committed rows through the path, the scan writes them back);
  // a scan-only verify needs the history CTAs of the commit kernel.
  fp.hist_in_kernels = prev_layers[0].x != nullptr && layers[0].x != nullptr;
  if (prev_layers[0].x && !fp.hist_in_kernels) {
    e = timed(ctx, LUMO_K_COMMIT, st, [&] {
      return launch_commit(ps, pt, fp.lb, accepted_dev, len_dev, lmax, false, true, pdl, st);
    });
    if (e != cudaSuccess) return cuda_fail(ctx, e, "history launch");
  }
  if (layers[0].x) {
    e = timed(ctx, LUMO_K_CONV, st, [&] {
      return fp.hist_in_kernels ? launch_conv_fused(s, t, lb, fp, pdl_conv, st) : launch_conv(s, t, lb, pdl_conv, st);
    });
    if (e != cudaSuccess) return cuda_fail(ctx, e, "conv launch");
  }
  e = timed(ctx, LUMO_K_SCAN, st, [&] {
    return ctx->scan_algo == 3 ? launch_scan_solve_fused(s, t, lb, fp, ctx->sm_count, pdl_scan, st)
                               : launch_scan_gram_fused(s, t, lb, fp, ctx->sm_count, pdl_scan, scan_tail(ctx, desc, s), st);
  });
  return e == cudaSuccess ? LUMO_OK : cuda_fail(ctx, e, "fused scan launch");
}

// ---- attention half ---------------------------------------------------------------------
namespace {

// Common checks of the three attention-side calls; fills the shape shared by all layers.
int prepare_attn(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_attn_args* layers, int n_layers, AttnShape* s) {
  if (!ctx || !desc || !layers) return fail(ctx, LUMO_ERR_ARG, "null ctx, desc or layers");
  if (desc->ctx != ctx) return fail(ctx, LUMO_ERR_ARG, "descriptor belongs to another context");
  if (ctx->device < 0) return fail(ctx, LUMO_ERR_UNSUPPORTED, "host-only context cannot launch");
  if (n_layers < 1 || n_layers > kMaxAttnLayers)
    return fail(ctx, LUMO_ERR_ARG, "n_layers must be in [1, " + std::to_string(kMaxAttnLayers) + "]");
  if (!desc->d_vis) return fail(ctx, LUMO_ERR_UNSUPPORTED, "the attention calls take at most 256 physical slots");
  const lumo_attn_args& a0 = layers[0];
  if (a0.dh != 128) return fail(ctx, LUMO_ERR_UNSUPPORTED, "dh must be 128");
  if (a0.Hq < 1 || a0.Hkv < 1 || a0.Hq % a0.Hkv != 0) return fail(ctx, LUMO_ERR_UNSUPPORTED, "Hq must be a positive multiple of Hkv");
  if (a0.Hkv > 32767) return fail(ctx, LUMO_ERR_UNSUPPORTED, "at most 32767 KV heads");
  if (!(a0.scale > 0.f)) return fail(ctx, LUMO_ERR_ARG, "scale must be positive");
  if (a0.n_cache_rows < 1 || a0.max_positions < desc->Ns)
    return fail(ctx, LUMO_ERR_ARG, "need n_cache_rows >= 1 and max_positions >= n_slots");
  if ((long long)a0.max_positions * a0.Hkv * a0.dh * 2 >= (1LL << 40))
    return fail(ctx, LUMO_ERR_UNSUPPORTED, "a cache row must span less than 2^40 bytes");
  if (!a0.ctx_len || !a0.cache_row) return fail(ctx, LUMO_ERR_ARG, "ctx_len and cache_row are required");
  // the kernels count key tiles of all (sequence, KV head, row tile) units in 32 bits
  if ((double)desc->B * a0.Hkv * attn_row_tiles(a0.Hq / a0.Hkv, desc->N) * ((double)a0.max_positions / 128 + 8) >= 2147483648.0)
    return fail(ctx, LUMO_ERR_UNSUPPORTED, "batch x KV heads x positions too large for one call");
  if (a0.kv_layout != 0 && a0.kv_layout != 1) return fail(ctx, LUMO_ERR_ARG, "kv_layout must be 0 or 1");
  if (a0.n_splits < 0 || a0.n_splits > 32) return fail(ctx, LUMO_ERR_ARG, "n_splits must be 0 (automatic) or in [1, 32]");
  for (int l = 0; l < n_layers; ++l) {
    const lumo_attn_args& a = layers[l];
    const std::string at = " (layer " + std::to_string(l) + ")";
    if (a.Hq != a0.Hq || a.Hkv != a0.Hkv || a.dh != a0.dh || a.scale != a0.scale || a.n_cache_rows != a0.n_cache_rows ||
        a.max_positions != a0.max_positions || a.ctx_len != a0.ctx_len || a.cache_row != a0.cache_row ||
        a.n_splits != a0.n_splits || a.kv_layout != a0.kv_layout)
      return fail(ctx, LUMO_ERR_ARG, "all layers must share shapes, options, ctx_len and cache_row" + at);
    if (!a.k_cache || !a.v_cache) return fail(ctx, LUMO_ERR_ARG, "k_cache and v_cache are required" + at);
    for (const void* p : {(const void*)a.k_cache, (const void*)a.v_cache, a.q, a.k_new, a.v_new, (const void*)a.out})
      if (p && !aligned16(p)) return fail(ctx, LUMO_ERR_ARG, "tensor pointers must be 16-byte aligned" + at);
  }
  s->B = desc->B; s->N = desc->N; s->Ns = desc->Ns; s->Hq = a0.Hq; s->Hkv = a0.Hkv;
  s->n_rows = a0.n_cache_rows; s->max_pos = a0.max_positions; s->scale = a0.scale;
  s->ctx_len = a0.ctx_len; s->cache_row = a0.cache_row;
  s->S = a0.n_splits;
  s->layout = a0.kv_layout;
  return LUMO_OK;
}

void kv_views(const lumo_tree_desc* desc, const lumo_attn_args* layers, int n_layers, const AttnShape& s, KvLayers* L, KvShape* k) {
  std::memset(L, 0, sizeof(*L));
  for (int l = 0; l < n_layers; ++l) {
    L->k[l] = layers[l].k_cache; L->v[l] = layers[l].v_cache;
    L->kn[l] = layers[l].k_new; L->vn[l] = layers[l].v_new;
    L->status[l] = layers[l].status;
  }
  k->B = s.B; k->N = s.N; k->Ns = s.Ns; k->Hkv = s.Hkv; k->n_rows = s.n_rows; k->max_pos = s.max_pos; k->layout = s.layout;
  k->ctx_len = s.ctx_len; k->cache_row = s.cache_row; k->parent = desc->d_parent; k->slot = desc->d_slot;
}

}  // namespace

int lumo_kv_write_tree(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_attn_args* layers, int n_layers, void* stream) {
  AttnShape s;
  int rc = prepare_attn(ctx, desc, layers, n_layers, &s);
  if (rc != LUMO_OK) return rc;
  for (int l = 0; l < n_layers; ++l)
    if (!layers[l].k_new || !layers[l].v_new) return fail(ctx, LUMO_ERR_ARG, "k_new and v_new are required");
  DeviceGuard g(ctx->device);
  cudaStream_t st = (cudaStream_t)stream;
  KvLayers L;
  KvShape k;
  kv_views(desc, layers, n_layers, s, &L, &k);
  cudaError_t e = cudaSuccess;
  for (int l = 0; l < n_layers && e == cudaSuccess; ++l)
    if (layers[l].status) e = cudaMemsetAsync(layers[l].status, 0, (size_t)s.B * sizeof(int32_t), st);
  if (e == cudaSuccess) e = timed(ctx, LUMO_K_KV_WRITE, st, [&] { return launch_kv_write(L, k, n_layers, st); });
  ctx->last_call = lumo_ctx::kOther;
  return e == cudaSuccess ? LUMO_OK : cuda_fail(ctx, e, "kv write launch");
}

int lumo_tree_attention(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_attn_args* layers, int n_layers, void* stream) {
  AttnShape s;
  int rc = prepare_attn(ctx, desc, layers, n_layers, &s);
  if (rc != LUMO_OK) return rc;
  for (int l = 0; l < n_layers; ++l)
    if (!layers[l].q || !layers[l].out) return fail(ctx, LUMO_ERR_ARG, "q and out are required");
  DeviceGuard g(ctx->device);
  cudaStream_t st = (cudaStream_t)stream;
  const size_t need = attn_scratch_bytes(s, ctx->sm_count);
  if (need > ctx->attn_scratch_bytes) {
    // first call with this shape: grow the scratch (synchronises; later calls allocate nothing)
    cudaError_t e = cudaSuccess;
    if (ctx->attn_scratch) {
      e = cudaDeviceSynchronize();
      if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaDeviceSynchronize");
      cudaFree(ctx->attn_scratch);
      ctx->attn_scratch = nullptr;
      ctx->attn_scratch_bytes = 0;
    }
    e = cudaMalloc(&ctx->attn_scratch, need);
    if (e != cudaSuccess) return fail(ctx, LUMO_ERR_NOMEM, std::string("scratch allocation failed: ") + cudaGetErrorString(e));
    ctx->attn_scratch_bytes = need;
    e = cudaMemset(ctx->attn_scratch, 0, 256);   // the failure flag in the first bytes: launch numbers are never 0
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaMemset(attention scratch)");
  }
  ctx->last_call = lumo_ctx::kOther;
  // the layers of a model are not adjacent in time: one launch (and one pair of tensor maps) per layer;
  // they share the scratch, which stream order makes safe
  for (int l = 0; l < n_layers; ++l) {
    AttnLayerPtrs p;
    p.k_cache = layers[l].k_cache; p.v_cache = layers[l].v_cache; p.q = layers[l].q;
    p.out = layers[l].out; p.lse = layers[l].lse; p.status = layers[l].status;
    AttnPlan plan;
    std::string err;
    if (++ctx->attn_launch_id == 0) ctx->attn_launch_id = 1;
    const uint32_t launch_id = ctx->attn_launch_id;
    cudaError_t e = attn_plan(s, p, desc->d_vis, desc->d_slot_used, reinterpret_cast<float*>(ctx->attn_scratch),
                              ctx->sm_count, launch_id, &plan, &err);
    if (e != cudaSuccess) return err.empty() ? cuda_fail(ctx, e, "attention set-up") : fail(ctx, LUMO_ERR_CUDA, err);
    e = timed(ctx, LUMO_K_ATTN, st, [&] { return launch_attn(plan, st); });
    if (e != cudaSuccess) return cuda_fail(ctx, e, "attention launch");
    e = timed(ctx, LUMO_K_ATTN_MERGE, st, [&] { return launch_attn_merge(plan, st); });
    if (e != cudaSuccess) return cuda_fail(ctx, e, "attention merge launch");
  }
  return LUMO_OK;
}

int lumo_kv_publish(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_attn_args* layers, int n_layers,
                    const int32_t* accepted_dev, const int32_t* len_dev, int lmax, int32_t* ctx_len_out, void* stream) {
  if (ctx && (lmax < 1 || lmax > kMaxNodes))
    return fail(ctx, LUMO_ERR_ARG, "lmax must be in [1, " + std::to_string(kMaxNodes) + "] (a path holds each node at most once)");
  AttnShape s;
  int rc = prepare_attn(ctx, desc, layers, n_layers, &s);
  if (rc != LUMO_OK) return rc;
  if (!accepted_dev || !len_dev) return fail(ctx, LUMO_ERR_ARG, "accepted_dev and len_dev are required");
  if (ctx_len_out == s.ctx_len) return fail(ctx, LUMO_ERR_ARG, "ctx_len_out must not alias ctx_len");
  DeviceGuard g(ctx->device);
  cudaStream_t st = (cudaStream_t)stream;
  KvLayers L;
  KvShape k;
  kv_views(desc, layers, n_layers, s, &L, &k);
  cudaError_t e = timed(ctx, LUMO_K_KV_PUBLISH, st, [&] {
    return launch_kv_publish(L, k, n_layers, accepted_dev, len_dev, lmax, ctx_len_out, st);
  });
  ctx->last_call = lumo_ctx::kOther;
  return e == cudaSuccess ? LUMO_OK : cuda_fail(ctx, e, "kv publish launch");
}

}  // extern "C"
