// Host-side tree descriptor: validation, integer tables and the scan schedule.
//
// Tables follow the paper's descriptor (parent indices, depth, logical<->physical slot
// maps; Sec. "State and the execution boundary") and its path-parallel schedule
// (dependent path groups, cut states; Sec. "Path-parallel verification and state
// lifetime").  The depth-first op list is this library's own schedule.
#include <algorithm>
#include <bitset>
#include <functional>

#include "internal.h"

namespace lumo {

namespace {

struct Kids {
  std::vector<int> root;
  std::vector<std::vector<int>> of;
};

// Depth-first op list.  `need_state(c)`: the node's state must be materialised (it has
// children, or every state is wanted for snapshots).  Returns the stack levels used.
int build_schedule(const Kids& kids, int N, const std::function<bool(int)>& need_state,
                   std::vector<int32_t>* ops) {
  int max_levels = 0;
  // recursion depth is bounded by the tree depth (<= 256)
  std::function<void(int, int)> visit = [&](int p, int lvl) {
    const std::vector<int>& ch = p < 0 ? kids.root : kids.of[p];
    std::vector<int> inner;
    for (int c : ch)
      if (need_state(c)) inner.push_back(c);
    if (inner.empty()) {
      for (int c : ch) ops->push_back(make_op(OP_EMIT, 0, c));
      return;
    }
    const int last = inner.back();
    for (int c : ch) {
      if (c == last) continue;
      ops->push_back(make_op(OP_EMIT, need_state(c) ? 1 : 0, c));
    }
    if (inner.size() > 1) {
      const bool at_root = p < 0;
      if (!at_root) {
        ops->push_back(make_op(OP_PUSH, 0, lvl));
        max_levels = std::max(max_levels, lvl + 1);
      }
      for (size_t j = 0; j + 1 < inner.size(); ++j) {
        ops->push_back(make_op(OP_DESCEND, 0, inner[j]));
        visit(inner[j], at_root ? lvl : lvl + 1);
        ops->push_back(make_op(OP_POP, 0, at_root ? kPopRoot : lvl));
      }
    }
    ops->push_back(make_op(OP_EMIT_DESCEND, 0, last));
    visit(last, lvl);
  };
  (void)N;
  visit(-1, 0);
  return max_levels;
}

}  // namespace

bool build_tree(const int32_t* parent, const int32_t* slot, int N, int Ns, HostTree* t,
                int* levels_lean, int* levels_full, std::string* err) {
  for (int i = 0; i < N; ++i) {
    if (parent[i] < -1 || parent[i] >= i) {
      *err = "parent[" + std::to_string(i) + "] = " + std::to_string(parent[i]) +
             " is not in {-1} U [0, i)";
      return false;
    }
  }
  auto& depth = t->tab[LUMO_TAB_DEPTH];
  depth.resize(N);
  for (int i = 0; i < N; ++i) depth[i] = parent[i] < 0 ? 1 : depth[parent[i]] + 1;

  Kids kids;
  kids.of.resize(N);
  for (int i = 0; i < N; ++i) (parent[i] < 0 ? kids.root : kids.of[parent[i]]).push_back(i);

  auto& n_child = t->tab[LUMO_TAB_N_CHILD];
  auto& is_leaf = t->tab[LUMO_TAB_IS_LEAF];
  auto& child_off = t->tab[LUMO_TAB_CHILD_OFF];
  auto& child_list = t->tab[LUMO_TAB_CHILD_LIST];
  auto& leaves = t->tab[LUMO_TAB_LEAVES];
  n_child.resize(N);
  is_leaf.resize(N);
  child_off.assign(1, 0);
  child_list.insert(child_list.end(), kids.root.begin(), kids.root.end());
  child_off.push_back((int32_t)child_list.size());
  for (int i = 0; i < N; ++i) {
    n_child[i] = (int32_t)kids.of[i].size();
    is_leaf[i] = kids.of[i].empty();
    if (is_leaf[i]) leaves.push_back(i);
    child_list.insert(child_list.end(), kids.of[i].begin(), kids.of[i].end());
    child_off.push_back((int32_t)child_list.size());
  }

  auto& path_off = t->tab[LUMO_TAB_PATH_OFF];
  auto& path_nodes = t->tab[LUMO_TAB_PATH_NODES];
  path_off.assign(1, 0);
  for (int lf : leaves) {
    size_t start = path_nodes.size();
    for (int c = lf; c >= 0; c = parent[c]) path_nodes.push_back(c);
    std::reverse(path_nodes.begin() + start, path_nodes.end());
    path_off.push_back((int32_t)path_nodes.size());
  }

  auto& win = t->tab[LUMO_TAB_ANC_WIN];
  win.resize((size_t)N * 4);
  for (int i = 0; i < N; ++i) {
    int cur = i, hist = 0;
    for (int j = 3; j >= 0; --j) {
      if (cur >= 0) { win[i * 4 + j] = cur; cur = parent[cur]; }
      else win[i * 4 + j] = -(++hist);
    }
  }

  auto& slot_inv = t->tab[LUMO_TAB_SLOT_INV];
  slot_inv.assign(Ns, -1);
  for (int i = 0; i < N; ++i) {
    int s = slot ? slot[i] : i;
    if (s < 0 || s >= Ns || slot_inv[s] != -1) {
      *err = "slot map is not injective into [0, n_slots) at node " + std::to_string(i);
      return false;
    }
    slot_inv[s] = i;
  }

  // attention visibility over the physical suffix: a node sees its own slot and what its parent sees
  if (Ns <= kMaxAttnSlots) {
    auto& vis = t->tab[LUMO_TAB_ATTN_VIS];
    const int W = (Ns + 31) / 32;
    vis.assign((size_t)N * W, 0);
    for (int i = 0; i < N; ++i) {
      if (parent[i] >= 0)
        for (int w = 0; w < W; ++w) vis[(size_t)i * W + w] = vis[(size_t)parent[i] * W + w];
      const int s = slot ? slot[i] : i;
      vis[(size_t)i * W + (s >> 5)] = (int32_t)((uint32_t)vis[(size_t)i * W + (s >> 5)] | (1u << (s & 31)));
    }
  }

  // chain decomposition: principal child = lowest index
  auto& c_head = t->tab[LUMO_TAB_CHAIN_HEAD];
  auto& c_off = t->tab[LUMO_TAB_CHAIN_OFF];
  auto& c_nodes = t->tab[LUMO_TAB_CHAIN_NODES];
  auto& c_level = t->tab[LUMO_TAB_CHAIN_LEVEL];
  auto& cut = t->tab[LUMO_TAB_CUT_NODES];
  std::vector<int> chain_of(N, -1);
  for (int i = 0; i < N; ++i)
    if (parent[i] < 0 || kids.of[parent[i]].front() != i) c_head.push_back(i);
  c_off.assign(1, 0);
  for (size_t c = 0; c < c_head.size(); ++c) {
    for (int cur = c_head[c];; cur = kids.of[cur].front()) {
      c_nodes.push_back(cur);
      chain_of[cur] = (int)c;
      if (kids.of[cur].empty()) break;
    }
    c_off.push_back((int32_t)c_nodes.size());
  }
  // heads ascend with their chain index and a head's parent lies in an earlier chain
  c_level.resize(c_head.size());
  std::vector<char> is_cut(N, 0);
  for (size_t c = 0; c < c_head.size(); ++c) {
    int p = parent[c_head[c]];
    c_level[c] = p < 0 ? 0 : c_level[chain_of[p]] + 1;
    if (p >= 0) is_cut[p] = 1;
  }
  for (int i = 0; i < N; ++i)
    if (is_cut[i]) cut.push_back(i);

  *levels_lean = build_schedule(kids, N, [&](int c) { return !kids.of[c].empty(); },
                                &t->tab[LUMO_TAB_SCHEDULE]);
  *levels_full = build_schedule(kids, N, [](int) { return true; }, &t->tab[LUMO_TAB_SCHEDULE_FULL]);
  return true;
}

// Node groups of the tensor-core scan.  A group is a set of at most 64 nodes closed under "parent
// of", so that it can be solved from the pre-tree state alone; every node is emitted (written) by
// exactly one group and may be recomputed, unwritten, in others.  Fewer groups mean fewer passes
// over the state, so the tree is first cut into atoms (a complete subtree if it fits together with
// its ancestors, else the node alone and its children in turn) and the atoms are packed, largest
// closure first, each into the group whose node set grows least (groups that already hold the
// atom's ancestors take it for little), or into a new group.  Members are ordered by (depth, index).
void build_gram_groups(const int32_t* parent, int N, const HostTree& t, std::vector<GramGroup>* out) {
  const auto& depth = t.tab[LUMO_TAB_DEPTH];
  const auto& coff = t.tab[LUMO_TAB_CHILD_OFF];
  const auto& clist = t.tab[LUMO_TAB_CHILD_LIST];
  constexpr int kCap = 64;
  using Mask = std::bitset<kMaxNodes>;
  std::vector<int> size(N, 1);
  for (int i = N - 1; i >= 0; --i)
    if (parent[i] >= 0) size[parent[i]] += size[i];
  struct Atom { Mask emit, closure; int count; };
  std::vector<Atom> atoms;
  // depth-first over the tree with an explicit stack (a = -1: children of the pre-tree state)
  std::vector<int> todo;
  for (int ci = coff[1] - 1; ci >= coff[0]; --ci) todo.push_back(clist[ci]);
  while (!todo.empty()) {
    const int c = todo.back();
    todo.pop_back();
    Atom at;
    if (size[c] + depth[c] - 1 <= kCap) {            // the whole subtree and its ancestors fit
      std::vector<int> st{c};
      while (!st.empty()) {
        const int n = st.back();
        st.pop_back();
        at.emit.set(n);
        for (int k = coff[n + 1]; k < coff[n + 2]; ++k) st.push_back(clist[k]);
      }
    } else {
      at.emit.set(c);
      for (int k = coff[c + 2] - 1; k >= coff[c + 1]; --k) todo.push_back(clist[k]);
    }
    at.closure = at.emit;
    for (int a = parent[c]; a >= 0; a = parent[a]) at.closure.set(a);
    at.count = (int)at.closure.count();
    atoms.push_back(at);
  }
  std::stable_sort(atoms.begin(), atoms.end(), [](const Atom& x, const Atom& y) { return x.count > y.count; });
  std::vector<Atom> bins;
  for (const Atom& at : atoms) {
    int best = -1, best_growth = 0;
    for (int b = 0; b < (int)bins.size(); ++b) {
      const int total = (int)(bins[b].closure | at.closure).count();
      if (total > kCap) continue;
      const int growth = total - bins[b].count;
      if (best < 0 || growth < best_growth) { best = b; best_growth = growth; }
    }
    if (best < 0) {
      bins.push_back(at);
    } else {
      bins[best].emit |= at.emit;
      bins[best].closure |= at.closure;
      bins[best].count = (int)bins[best].closure.count();
    }
  }
  for (const Atom& bin : bins) {
    GramGroup g;
    std::vector<int> all;
    for (int n = 0; n < N; ++n)
      if (bin.closure.test(n)) all.push_back(n);
    std::sort(all.begin(), all.end(), [&](int x, int y) { return depth[x] != depth[y] ? depth[x] < depth[y] : x < y; });
    for (int n : all) {
      g.nodes.push_back(n);
      g.emit.push_back(bin.emit.test(n) ? 1 : 0);
    }
    out->push_back(std::move(g));
  }
}

}  // namespace lumo
