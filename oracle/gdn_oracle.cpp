// fp64 CPU oracle for the GDN tree verify + commit path.
//
// TEST INFRASTRUCTURE ONLY.  Plain, slow, written from the paper's definitions; it
// shares no code with the CUDA library and is never on the product path.  Only the
// tests, the smoke check and the benchmark's CPU-baseline leg call it.
//
// What it computes, per sequence b and value head h (q/k head g = h / (Hv/Hk)):
//
//  * oracle_conv   - the ancestry-gathered causal depthwise convolution (width 4) and
//                    SiLU (Sec. "Precompute branch histories while preserving
//                    arithmetic": windows are gathered from the prior convolution
//                    history and the candidate inputs along each node's ancestry;
//                    taps are applied in order, oldest first; one cast at the end).
//  * oracle_scan   - the recurrence of Eq. 2-3 for every node of the tree, starting
//                    from the pre-tree state and walking the node's ancestry root
//                    first:  R' = alpha R_parent;  delta = beta (v - R' k);
//                    R = R' + delta k^T;  o = R q.   R is d_v x d_k.
//                    "walk" mode recomputes every node from the root state (the
//                    definition); "memo" mode caches each parent's state (the same
//                    operations in the same order per node, so bitwise equal).
//  * oracle_commit - Algorithm 2, "Replay only the accepted path into native
//                    recurrent state": start from the pre-tree state, apply the same
//                    update for the accepted nodes in path order, publish in place;
//                    and Algorithm 1 line "Gather the convolution history for A into
//                    the native running row".
//
// Pins (tests/test_oracle_*.py): a chain equals the textbook sequential gated delta
// rule and a library causal conv1d; beta = 0 gives pure decay; alpha = 1, beta = 0
// leaves the state bitwise unchanged; walk == memo bitwise; the retrieval invariant
// S_i k_i = (1-beta) alpha S_p k_i + beta v_i; orthonormal keys overwrite single
// columns; an ancestor-masked triangular solve with a library routine; an independent
// NumPy restatement; off-path poisoning and slot permutation leave results bitwise
// unchanged.  The paper prints no worked numeric example, so absolute values are
// pinned only through those identities.
//
// Build: g++ -O2 -ffp-contract=off -shared -fPIC (no fast-math: the walk/memo bitwise
// pin and the alpha = 1, beta = 0 pin depend on plain IEEE double arithmetic).
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>
#include <algorithm>

namespace {

// Round a double to the nearest bfloat16 (ties to even), returned as a double.
double round_bf16(double x) {
  if (!std::isfinite(x) || x == 0.0) return x;
  int e;
  std::frexp(x, &e);            // |x| = m 2^e, m in [0.5, 1)  ->  floor(log2|x|) = e - 1
  int ex = e - 1;
  if (ex < -126) ex = -126;     // subnormal range shares the smallest normal's spacing
  double ulp = std::ldexp(1.0, ex - 7);   // 8 significand bits
  double y = std::nearbyint(x / ulp) * ulp;  // division by a power of two is exact; RNE
  const double max_bf16 = 3.3895313892515355e38;  // (2 - 2^-7) 2^127
  if (std::fabs(y) > max_bf16) y = std::copysign(INFINITY, x);
  return y;
}

double round_to(double x, int dtype) {  // 0 = f32, 1 = bf16, 2 = keep fp64
  if (dtype == 0) return (double)(float)x;
  if (dtype == 1) return round_bf16(x);
  return x;
}

// Root-first ancestry of node i.
std::vector<int> ancestry(const int32_t* parent, int i) {
  std::vector<int> a;
  while (i >= 0) { a.push_back(i); i = parent[i]; }
  std::reverse(a.begin(), a.end());
  return a;
}

int n_threads(int requested, int jobs) {
  int t = requested > 0 ? requested : (int)std::thread::hardware_concurrency();
  if (t < 1) t = 1;
  return std::min(t, std::max(jobs, 1));
}

template <class F>
int parallel_for(int jobs, int requested, F f) {
  int nt = n_threads(requested, jobs);
  if (nt == 1) { for (int j = 0; j < jobs; ++j) f(j); return 1; }
  std::vector<std::thread> th;
  for (int t = 0; t < nt; ++t)
    th.emplace_back([=] { for (int j = t; j < jobs; j += nt) f(j); });
  for (auto& x : th) x.join();
  return nt;
}

// q/k preparation: optional L2 normalisation x / sqrt(sum x^2 + eps), then scale on q.
void prep_qk(const double* src, int d, int l2norm, double eps, double scale, double* dst) {
  double inv = 1.0;
  if (l2norm) {
    double ss = 0.0;
    for (int j = 0; j < d; ++j) ss += src[j] * src[j];
    inv = 1.0 / std::sqrt(ss + eps);
  }
  for (int j = 0; j < d; ++j) dst[j] = src[j] * inv * scale;
}

// One node update on a d x d state (row = value index, column = key index), Eq. 2-3.
void gdn_update(double* S, int d, double alpha, double beta, const double* k, const double* v) {
  for (int i = 0; i < d * d; ++i) S[i] = alpha * S[i];            // R' = alpha R_parent
  for (int r = 0; r < d; ++r) {
    double u = 0.0;
    for (int j = 0; j < d; ++j) u += S[r * d + j] * k[j];        // (R' k)_r
    double dl = beta * (v[r] - u);                                // delta_r
    for (int j = 0; j < d; ++j) S[r * d + j] += dl * k[j];       // R = R' + delta k^T
  }
}

void gdn_output(const double* S, int d, const double* q, double* o) {
  for (int r = 0; r < d; ++r) {
    double acc = 0.0;
    for (int j = 0; j < d; ++j) acc += S[r * d + j] * q[j];      // o = R q
    o[r] = acc;
  }
}

int check_path(const int32_t* parent, int N, const int32_t* acc, int len, int lmax) {
  if (len < 0 || len > lmax) return 1;
  for (int t = 0; t < len; ++t) {
    int a = acc[t];
    if (a < 0 || a >= N) return 2;
    if (t == 0) { if (parent[a] != -1) return 3; }
    else if (parent[a] != acc[t - 1]) return 4;
  }
  return 0;
}

}  // namespace

extern "C" {

// x [B,Ns,C]; w [C,4]; bias [C] or null; hist [rows,3,C] oldest first; y [B,Ns,C] (physical
// rows; padding rows and skipped sequences are zero).  out_dtype: 0 f32, 1 bf16, 2 none.
int oracle_conv(int B, int N, int Ns, int C, const int32_t* parent, const int32_t* slot,
                const int32_t* state_row, const double* x, const double* w, const double* bias,
                const double* hist, int out_dtype, double* y, int threads) {
  std::memset(y, 0, sizeof(double) * (size_t)B * Ns * C);
  return parallel_for(B * N, threads, [&](int job) {
    int b = job / N, i = job % N;
    int row = state_row[b];
    if (row < 0) return;
    const int32_t* par = parent + (size_t)b * N;
    const int32_t* sl = slot + (size_t)b * N;
    // window: entry 3 = node, 2 = parent, 1 = grandparent, 0 = great-grandparent; past R the
    // walk continues into the committed history, most recent row first.
    const double* src[4];
    int cur = i, used_hist = 0;
    for (int j = 3; j >= 0; --j) {
      if (cur >= 0) {
        src[j] = x + ((size_t)b * Ns + sl[cur]) * C;
        cur = par[cur];
      } else {
        ++used_hist;                                   // 1 = most recent = hist row 2
        src[j] = hist + ((size_t)row * 3 + (3 - used_hist)) * C;
      }
    }
    double* out = y + ((size_t)b * Ns + sl[i]) * C;
    for (int c = 0; c < C; ++c) {
      double acc = 0.0;
      for (int j = 0; j < 4; ++j) acc += w[(size_t)c * 4 + j] * src[j][c];   // oldest -> newest
      if (bias) acc += bias[c];
      double s = acc / (1.0 + std::exp(-acc));          // SiLU
      out[c] = round_to(s, out_dtype);
    }
  });
}

// q,k [B,Ns,Hk,d]; v [B,Ns,Hv,d]; alpha,beta [B,Ns,Hv]; state pool [rows,Hv,d,d];
// o [B,Ns,Hv,d]; snap_nodes [B,E] logical ids (-1 = none) -> snap [B,E,Hv,d,d] (may be null).
// mode 0 = walk (definition), 1 = memo.
int oracle_scan(int B, int N, int Ns, int Hk, int Hv, int d, const int32_t* parent,
                const int32_t* slot, const int32_t* state_row, const double* q, const double* k,
                const double* v, const double* alpha, const double* beta, const double* state,
                double scale, int l2norm, double eps, int mode, double* o,
                const int32_t* snap_nodes, int E, double* snap, int threads) {
  std::memset(o, 0, sizeof(double) * (size_t)B * Ns * Hv * d);
  if (snap) std::memset(snap, 0, sizeof(double) * (size_t)B * E * Hv * d * d);
  const int rep = Hv / Hk;
  return parallel_for(B * Hv, threads, [&](int job) {
    int b = job / Hv, h = job % Hv, g = h / rep;
    int row = state_row[b];
    if (row < 0) return;
    const int32_t* par = parent + (size_t)b * N;
    const int32_t* sl = slot + (size_t)b * N;
    const double* S0 = state + ((size_t)row * Hv + h) * d * d;
    // prepared operands per logical node
    std::vector<double> qn((size_t)N * d), kn((size_t)N * d);
    for (int i = 0; i < N; ++i) {
      size_t pr = (size_t)b * Ns + sl[i];
      prep_qk(q + (pr * Hk + g) * d, d, l2norm, eps, scale, &qn[(size_t)i * d]);
      prep_qk(k + (pr * Hk + g) * d, d, l2norm, eps, 1.0, &kn[(size_t)i * d]);
    }
    auto node_v = [&](int i) { return v + (((size_t)b * Ns + sl[i]) * Hv + h) * d; };
    auto node_a = [&](int i) { return alpha[((size_t)b * Ns + sl[i]) * Hv + h]; };
    auto node_b = [&](int i) { return beta[((size_t)b * Ns + sl[i]) * Hv + h]; };
    auto emit = [&](int i, const double* S) {
      gdn_output(S, d, &qn[(size_t)i * d], o + (((size_t)b * Ns + sl[i]) * Hv + h) * d);
      if (snap)
        for (int e = 0; e < E; ++e)
          if (snap_nodes[(size_t)b * E + e] == i)
            std::memcpy(snap + (((size_t)b * E + e) * Hv + h) * d * d, S, sizeof(double) * d * d);
    };
    if (mode == 0) {
      std::vector<double> S((size_t)d * d);
      for (int i = 0; i < N; ++i) {
        std::memcpy(S.data(), S0, sizeof(double) * d * d);
        for (int t : ancestry(par, i))
          gdn_update(S.data(), d, node_a(t), node_b(t), &kn[(size_t)t * d], node_v(t));
        emit(i, S.data());
      }
    } else {
      std::vector<std::vector<double>> st(N);
      for (int i = 0; i < N; ++i) {     // parent[i] < i: parents are ready
        const double* Sp = par[i] < 0 ? S0 : st[par[i]].data();
        st[i].assign(Sp, Sp + (size_t)d * d);
        gdn_update(st[i].data(), d, node_a(i), node_b(i), &kn[(size_t)i * d], node_v(i));
        emit(i, st[i].data());
      }
    }
  });
}

// In place on `state` [rows,Hv,d,d] and (if x != null) `hist` [rows,3,C].  accepted [B,lmax]
// logical ids root first; len [B].  status [B] receives 0 or the first failed check; a failed
// sequence is left untouched.  x [B,Ns,C] raw pre-conv inputs.
int oracle_commit(int B, int N, int Ns, int Hk, int Hv, int d, const int32_t* parent,
                  const int32_t* slot, const int32_t* state_row, const double* q, const double* k,
                  const double* v, const double* alpha, const double* beta, double* state,
                  double scale, int l2norm, double eps, const int32_t* accepted,
                  const int32_t* len, int lmax, const double* x, int C, double* hist,
                  int32_t* status, int threads) {
  (void)scale;  // the query scale does not enter the state update
  const int rep = Hv / Hk;
  for (int b = 0; b < B; ++b) {
    status[b] = 0;
    if (state_row[b] < 0) continue;
    status[b] = check_path(parent + (size_t)b * N, N, accepted + (size_t)b * lmax, len[b], lmax);
  }
  int used = parallel_for(B * Hv, threads, [&](int job) {
    int b = job / Hv, h = job % Hv, g = h / rep;
    int row = state_row[b];
    if (row < 0 || status[b] != 0) return;
    const int32_t* sl = slot + (size_t)b * N;
    double* S = state + ((size_t)row * Hv + h) * d * d;
    std::vector<double> kn(d);
    for (int t = 0; t < len[b]; ++t) {
      int i = accepted[(size_t)b * lmax + t];
      size_t pr = (size_t)b * Ns + sl[i];
      prep_qk(k + (pr * Hk + g) * d, d, l2norm, eps, 1.0, kn.data());
      gdn_update(S, d, alpha[pr * Hv + h], beta[pr * Hv + h], kn.data(), v + (pr * Hv + h) * d);
    }
  });
  if (x && hist) {
    for (int b = 0; b < B; ++b) {
      int row = state_row[b];
      if (row < 0 || status[b] != 0) continue;
      const int32_t* sl = slot + (size_t)b * N;
      // last three rows of [old history ; x of the accepted nodes]
      std::vector<const double*> seq;
      std::vector<double> old((size_t)3 * C);
      std::memcpy(old.data(), hist + (size_t)row * 3 * C, sizeof(double) * 3 * C);
      for (int j = 0; j < 3; ++j) seq.push_back(&old[(size_t)j * C]);
      for (int t = 0; t < len[b]; ++t)
        seq.push_back(x + ((size_t)b * Ns + sl[accepted[(size_t)b * lmax + t]]) * C);
      for (int j = 0; j < 3; ++j)
        std::memcpy(hist + ((size_t)row * 3 + j) * C, seq[seq.size() - 3 + j], sizeof(double) * C);
    }
  }
  return used;
}

double oracle_round_bf16(double x) { return round_bf16(x); }

}  // extern "C"
