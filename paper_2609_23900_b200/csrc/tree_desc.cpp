// Host-side tree descriptor: validation, integer tables and the scan schedule.
//
// Tables follow the paper's descriptor (parent indices, depth, logical<->physical slot
// maps; Sec. "State and the execution boundary") and its path-parallel schedule
// (dependent path groups, cut states; Sec. "Path-parallel verification and state
// lifetime").  The depth-first op list is this library's own schedule.
#include <algorithm>
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

// Partition of a tree into groups of at most 64 nodes for the Gram-form scan.  A group is a
// root-first prefix path (whose deltas the group recomputes) plus complete subtrees hanging off
// the last prefix node, so every member's ancestors are inside the group.  A node is emitted
// (its output written) by exactly one group: as a subtree member, or by the first group that
// carries it as a prefix node.  Members are ordered by (depth, logical index).
void build_gram_groups(const int32_t* parent, int N, const HostTree& t, std::vector<GramGroup>* out) {
  const auto& depth = t.tab[LUMO_TAB_DEPTH];
  const auto& coff = t.tab[LUMO_TAB_CHILD_OFF];
  const auto& clist = t.tab[LUMO_TAB_CHILD_LIST];
  std::vector<int> size(N, 1);
  for (int i = N - 1; i >= 0; --i)
    if (parent[i] >= 0) size[parent[i]] += size[i];
  std::vector<char> emitted(N, 0);
  constexpr int kCap = 64;
  auto kids = [&](int a, int* lo, int* hi) { *lo = coff[a + 1]; *hi = coff[a + 2]; };   // a = -1: children of the pre-tree state
  auto flush = [&](const std::vector<int>& prefix, std::vector<int>& members) {
    if (members.empty()) return;
    GramGroup g;
    std::vector<int> all(prefix);
    all.insert(all.end(), members.begin(), members.end());
    std::sort(all.begin(), all.end(), [&](int x, int y) { return depth[x] != depth[y] ? depth[x] < depth[y] : x < y; });
    for (int n : all) {
      g.nodes.push_back(n);
      g.emit.push_back(emitted[n] ? 0 : 1);
      emitted[n] = 1;
    }
    out->push_back(std::move(g));
    members.clear();
  };
  std::function<void(int, std::vector<int>&)> pack = [&](int a, std::vector<int>& prefix) {
    const int cap = kCap - (int)prefix.size();
    int lo, hi;
    kids(a, &lo, &hi);
    std::vector<int> cur;
    for (int ci = lo; ci < hi; ++ci) {
      const int c = clist[ci];
      if (size[c] <= cap) {
        if ((int)cur.size() + size[c] > cap) flush(prefix, cur);
        // whole subtree of c (its nodes have indices > c; walk by parent marks)
        std::vector<int> stack{c};
        while (!stack.empty()) {
          int n = stack.back(); stack.pop_back();
          cur.push_back(n);
          int l2, h2;
          kids(n, &l2, &h2);
          for (int k = l2; k < h2; ++k) stack.push_back(clist[k]);
        }
      } else {
        flush(prefix, cur);
        prefix.push_back(c);
        pack(c, prefix);
        prefix.pop_back();
      }
    }
    flush(prefix, cur);
    if (a >= 0 && !emitted[a]) {      // every child was too large and recursed, or a has no group yet
      std::vector<int> none;
      GramGroup g;
      for (int n : prefix) { g.nodes.push_back(n); g.emit.push_back(emitted[n] ? 0 : 1); emitted[n] = 1; }
      out->push_back(std::move(g));
    }
  };
  std::vector<int> prefix;
  pack(-1, prefix);
}

}  // namespace lumo
