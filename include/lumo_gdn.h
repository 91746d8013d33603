/* lumo_gdn.h - C ABI of the B200 (sm_100a) Gated DeltaNet tree verifier and committer.
 *
 * The library verifies every node of a speculative candidate tree through one Gated
 * DeltaNet (GDN) layer and later replays the accepted path into the running state:
 *
 *   tree conv   y_i = SiLU(sum_j w[:,j] * x_{anc(i,3-j)})            (ancestry-gathered, width 4)
 *   tree scan   R'_i = alpha_i R_parent(i);  delta_i = beta_i (v_i - R'_i k_i);
 *               R_i = R'_i + delta_i k_i^T;  o_i = R_i q_i           (paper Eq. 2-3)
 *   commit      the same update for the accepted nodes in path order, published in place,
 *               plus the matching convolution history             (paper Algorithms 1 and 2)
 *
 * Around these: lumo_gdn_commit_verify (the commit of the previous cycle folded into the next
 * verify), lumo_tree_accept (device-resident acceptance walk between verify and commit),
 * lumo_select_spine_top3 (fused draft selection upstream of the tree), lumo_gdn_tree_scan_static
 * (the scan with library-internal static scratch), the attention half of the same cycle
 * (lumo_kv_write_tree, lumo_tree_attention, lumo_kv_publish: the tree's KV entries written, read and
 * re-linearised through the same slot map) and small helpers.
 *
 * Conventions
 *   - One GPU.  All tensor pointers are DEVICE pointers owned by the caller unless a
 *     comment says HOST; the library never frees or reallocates caller memory.
 *   - Row-major, innermost dimension contiguous.  B = batch, N = logical nodes per tree,
 *     Ns >= N physical rows (padding), Hk q/k heads, Hv value heads (Hv % Hk == 0, value head
 *     h uses q/k head h / (Hv/Hk)), d = d_k = d_v in {64, 128}, C = 2 Hk d + Hv d channels.
 *   - Every per-node tensor is indexed by PHYSICAL row slot[b][i]; padding rows are never
 *     read and their outputs are written as zeros.
 *   - verify/commit/path_from_node only enqueue work on `stream` (a cudaStream_t passed as
 *     void*); they never synchronise.  They may grow library-owned scratch on the first call
 *     with a given shape; after that they allocate nothing.
 *   - Host-detectable problems return a non-zero lumo_status and enqueue nothing;
 *     lumo_last_error() then describes the problem.  Problems only the device can see are
 *     reported per sequence in the `status` words (lumo_seq_status) and leave that sequence's
 *     state and history untouched.  Kernels never trap and contain only bounded loops.
 */
#ifndef LUMO_GDN_H_
#define LUMO_GDN_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lumo_ctx lumo_ctx;             /* device id + library-owned scratch */
typedef struct lumo_tree_desc lumo_tree_desc; /* host + device copies of the topology tables */

typedef enum {
  LUMO_OK = 0,
  LUMO_ERR_ARG = 1,         /* null / out-of-range argument */
  LUMO_ERR_TREE = 2,        /* parent array or slot map violates the rules below */
  LUMO_ERR_PATH = 3,        /* reserved for host-side path checks */
  LUMO_ERR_UNSUPPORTED = 4, /* shape or dtype outside the supported set */
  LUMO_ERR_CUDA = 5,        /* a CUDA runtime call failed */
  LUMO_ERR_NOMEM = 6        /* scratch allocation failed */
} lumo_status;

typedef enum { LUMO_F32 = 0, LUMO_BF16 = 1 } lumo_dtype;

/* Per-sequence device status words (first failing check wins, in this order). */
typedef enum {
  LUMO_SEQ_OK = 0,
  LUMO_SEQ_BAD_LEN = 1,   /* accepted length < 0 or > lmax (or path longer than lmax) */
  LUMO_SEQ_BAD_NODE = 2,  /* accepted entry outside [0, N) */
  LUMO_SEQ_BAD_ROOT = 3,  /* first accepted entry is not a child of the pre-tree state */
  LUMO_SEQ_BAD_LINK = 4,  /* accepted entry t is not a child of entry t-1 */
  LUMO_SEQ_BAD_ROW = 5,   /* state_row[b] >= n_state_rows */
  LUMO_SEQ_TIMEOUT = 6,   /* a bounded device-side wait ran out; outputs of the call are invalid */
  LUMO_SEQ_BAD_CTX = 7    /* attention calls: ctx_len[b] < 0 or ctx_len[b] + Ns > max_positions */
} lumo_seq_status;

/* Integer tables of one tree (lumo_tree_desc_get).  The paper's tree descriptor holds parent
 * indices, depth and the logical<->physical maps (Sec. "State and the execution boundary");
 * the path tables are what its path-parallel schedule is built from (Sec. "Path-parallel
 * verification and state lifetime").  All answers are unique. */
typedef enum {
  LUMO_TAB_DEPTH = 0,      /* [N]   1 + depth[parent]; a child of the pre-tree state has depth 1 */
  LUMO_TAB_N_CHILD = 1,    /* [N] */
  LUMO_TAB_CHILD_OFF = 2,  /* [N+2] CSR offsets: entry 0 = pre-tree state, entry i+1 = node i */
  LUMO_TAB_CHILD_LIST = 3, /* [N]   children in ascending logical index */
  LUMO_TAB_IS_LEAF = 4,    /* [N] */
  LUMO_TAB_LEAVES = 5,     /* [P]   ascending */
  LUMO_TAB_PATH_OFF = 6,   /* [P+1] CSR offsets of root-to-leaf paths */
  LUMO_TAB_PATH_NODES = 7, /*       root-first node list of each path */
  LUMO_TAB_ANC_WIN = 8,    /* [N*4] conv window: entry 3 = node, 2 = parent, ...; past the
                                     pre-tree state -1/-2/-3 = most recent / 2nd / 3rd history row */
  LUMO_TAB_SLOT_INV = 9,   /* [Ns]  logical node of each physical row, -1 = padding */
  LUMO_TAB_CHAIN_HEAD = 10,  /* chain decomposition: a chain starts at each child of the pre-tree */
  LUMO_TAB_CHAIN_OFF = 11,   /* state and at each non-lowest-index child and follows lowest-index */
  LUMO_TAB_CHAIN_NODES = 12, /* children to a leaf; level 0 = starts at the pre-tree state, else  */
  LUMO_TAB_CHAIN_LEVEL = 13, /* 1 + level of the chain holding the head's parent                  */
  LUMO_TAB_CUT_NODES = 14,   /* parents (not the pre-tree state) of chain heads, ascending, unique */
  LUMO_TAB_SCHEDULE = 15,    /* depth-first op list the scan kernel interprets, (kind<<24)|(flag<<20)|arg:
                                kind 0 EMIT node (output from the parent's state; flag: keep delta on
                                chip), 1 EMIT_DESCEND node (then turn the registers into the node's
                                state), 2 DESCEND node (same, from the kept delta), 3 PUSH level,
                                4 POP level (0xFFFF = reload the pre-tree state) */
  LUMO_TAB_SCHEDULE_FULL = 16, /* same, materialising every node's state (snapshot modes) */
  LUMO_TAB_GRAM_GROUPS = 17,   /* node groups of the tensor-core scan (empty if depth > 16): [G, then per
                                  group: n, n node ids ordered by (depth, index), n emit flags].  A group
                                  holds at most 64 nodes and every ancestor of each member; each node is
                                  emitted by exactly one group */
  LUMO_TAB_ATTN_VIS = 18,      /* [N, ceil(Ns/32)] attention visibility over the physical suffix: bit s of word s/32
                                  of node i is set when slot s holds i or an ancestor of i (32-bit patterns stored
                                  as int32); empty when Ns > 256, and then the attention calls are refused */
  LUMO_TAB_COUNT = 19
} lumo_table;

/* ---- context ------------------------------------------------------------------------- */
/* Creates a context on CUDA device `device`.  Returns LUMO_ERR_CUDA if no usable device.
 * device = -1 creates a host-only context: descriptors can be built and their integer tables
 * read, but every call that would launch returns LUMO_ERR_UNSUPPORTED (there is no CPU path). */
int lumo_ctx_create(int device, lumo_ctx** out);
void lumo_ctx_destroy(lumo_ctx* ctx);
/* Text of the last error recorded on this context (ctx-owned, valid until the next call);
 * with ctx == NULL, the last error of a failed lumo_ctx_create on this thread. */
const char* lumo_last_error(const lumo_ctx* ctx);
/* Bytes of library-owned device scratch currently held (for reporting). */
int64_t lumo_ctx_scratch_bytes(const lumo_ctx* ctx);

/* Which scan kernel lumo_gdn_tree_verify uses: 0 = automatic (the tensor-core kernel when the shape
 * allows it: d = 128, bf16 operands, tree depth <= 16, no snapshots; trees of more than 64 nodes are
 * cut into node groups on the host; else rank-1), 1 = always the rank-1 fp32 kernel, 2 = the Gram form
 * with a forward substitution over value rows, level by level, 3 = the solved Gram form (the triangular
 * system is solved on scalars per head and the state enters a single product with "effective queries"),
 * 4 = the Gram form with a closed-form tail (the same two products as 2; then M = W (I + A)^-1 by a back
 * substitution per node along its own root path and one pass that sums M x right-hand sides: no step
 * waits for another node), 5 = the closed form of 4 with that sum as one more tensor-core product over all
 * nodes of a group (right-hand sides and coefficients as bf16 hi + lo: relative 2^-16 on the sum; a right-hand
 * side that is not finite is kept out of the product and turns the outputs of its own subtree into NaN, as the
 * recurrence would).  "Automatic" picks between 2 and 5 per descriptor and launch (thin deep trees, a spine with
 * small side branches, take 5; other trees take 5 in launches of several waves where it measured faster; the
 * rest take 2).  2 to 5 return LUMO_ERR_UNSUPPORTED on other shapes. */
int lumo_ctx_set_scan_algo(lumo_ctx* ctx, int algo);

/* Test aid for the failure path of the tensor-core scan.  That kernel waits for its tensor-core work
 * on an mbarrier with a bounded number of polls; when the bound runs out it writes LUMO_SEQ_TIMEOUT
 * into the status words, frees its tensor memory and returns.  With the drill on, the kernel issues
 * no tensor-core work at all (so nothing asynchronous is in flight) and polls only 1024 times: the
 * wait runs out by construction and the failure path executes, harmlessly.  Outputs of such a call are
 * undefined.  Default off. */
int lumo_ctx_set_timeout_drill(lumo_ctx* ctx, int on);

/* Kernel overlap (default on): conv, scan and commit are launched with programmatic dependent launch,
 * so each kernel's set-up (and, for commit, its whole read phase) runs under the tail of the kernel
 * before it; each waits on the device before touching data its predecessor produces or still reads.
 * Applied only to small launches (n_layers * B * Hv <= 4 x SM count), where it measured faster.
 * Results are identical either way; 0 restores plain stream order.
 * The commit (and a scan without convolution) reads part of its input ahead of that wait: the
 * accepted path, the recorded operands, the state.  The library therefore overlaps it only when the
 * previous call on this context was a verify; behind any other library call it runs in plain stream
 * order.  A caller that fills accepted_dev / len_dev with a kernel of its own between verify and
 * commit, on the same stream, switches overlap off. */
int lumo_ctx_set_overlap(lumo_ctx* ctx, int on);

/* Measurement aid.  While enabled, every kernel the library launches is bracketed by two CUDA
 * events on the launch stream (up to 16384 launches between reads; later ones go untimed).
 * lumo_ctx_timing_read waits for the recorded events, returns the launch count and summed
 * device time of kernels of `kind` (lumo_kernel_kind) and, with reset != 0, forgets all
 * records.  Enabling allocates the event pool; do not enable inside a stream capture. */
typedef enum { LUMO_K_CONV = 0, LUMO_K_SCAN = 1, LUMO_K_COMMIT = 2, LUMO_K_PATH = 3,
               LUMO_K_ATTN = 4, LUMO_K_ATTN_MERGE = 5, LUMO_K_KV_WRITE = 6, LUMO_K_KV_PUBLISH = 7,
               LUMO_K_COUNT = 8 } lumo_kernel_kind;
int lumo_ctx_timing_enable(lumo_ctx* ctx, int enable);
int lumo_ctx_timing_read(lumo_ctx* ctx, int kind, int reset, int64_t* launches, double* total_ms);

/* ---- tree descriptor -------------------------------------------------------------------
 * parent, depth, slot are HOST arrays, copied.  parent[b*N+i] in {-1} U [0, i): -1 is the
 * pre-tree state ("a previous node in the packed buffer need not be the parent", Sec. "The
 * recurrence and path locality"; several children of -1 are allowed).  depth may be NULL
 * (derived) and is validated if given.  slot may be NULL (identity) and must otherwise be
 * injective into [0, n_slots).  1 <= N <= 256, N <= n_slots <= 1024.
 * Errors: LUMO_ERR_ARG, LUMO_ERR_TREE, LUMO_ERR_CUDA.  May synchronise (host-to-device copy). */
int lumo_tree_desc_create(lumo_ctx* ctx, int batch, int n_nodes, int n_slots,
                          const int32_t* parent, const int32_t* depth, const int32_t* slot,
                          lumo_tree_desc** out);
void lumo_tree_desc_destroy(lumo_tree_desc* desc);
/* HOST copy of table `which` (lumo_table) of sequence b; desc-owned memory. */
int lumo_tree_desc_get(const lumo_tree_desc* desc, int which, int b, const int32_t** data,
                       int64_t* count);
/* Device helper (Sec. "One device-selected path drives native continuation": accepted node
 * indices and path lengths are fixed-shape device products): for every sequence, the root-first
 * node list of the path that ends at node_dev[b] (-1 = empty path) -> accepted_dev [B, lmax]
 * (-1 padded), len_dev [B]; status_dev [B] (may be NULL) receives LUMO_SEQ_BAD_NODE /
 * LUMO_SEQ_BAD_LEN, in which case the path is written as empty. */
int lumo_tree_path_from_node(lumo_ctx* ctx, const lumo_tree_desc* desc, const int32_t* node_dev,
                             int lmax, int32_t* accepted_dev, int32_t* len_dev,
                             int32_t* status_dev, void* stream);

/* ---- acceptance walk ---------------------------------------------------------------------
 * The step between verify and commit (paper Algorithm 1, "Select one continuation": the accepted
 * materialized path and the pending token from sampling with the target probabilities p and the
 * proposal probabilities q; Sec. "One device-selected path drives native continuation": accepted
 * node indices, path lengths, emitted tokens and the selected final row are device products).
 * Starting at the pre-tree state the walk tries the children of the current node in ascending
 * logical index.  mode 0, greedy: the child whose token equals argmax of the current target row is
 * accepted (lowest token index on ties); otherwise the walk stops and the pending token is that
 * argmax.  mode 1, rejection sampling (accepted mass min(p, q), residual mass proportional to
 * (p - q)+, Appendix "Serving configuration and measurement"): child c with token x is accepted iff
 * u_c q_c(x) < r(x) / Z with r the unnormalised residual target (p at first), Z its sum; a rejection
 * replaces r by (r - Z q_c)+; when no child is accepted the pending token is argmax_i r_i / e_i over
 * the caller's Exp(1) variates (an exact draw from r / Z), lowest index on ties.  All device pointers. */
typedef struct {
  int32_t V;               /* vocabulary size */
  int32_t mode;            /* 0 greedy, 1 rejection sampling */
  const int32_t* token;    /* [B, Ns] candidate token of each physical row */
  const float* p_target;   /* [B, Ns+1, V] target probabilities after the node in physical row s;
                              row Ns: after the pre-tree state */
  const float* q_draft;    /* [B, Ns, V] proposal distribution the row's token was drawn from (mode 1) */
  const float* uniforms;   /* [B, Ns] one U[0,1) number per physical row (mode 1) */
  const float* noise;      /* [B, V] Exp(1) variates for the pending-token draw (mode 1) */
  float* work;             /* [B, V] scratch for the residual (mode 1); contents undefined afterwards */
} lumo_accept_args;
/* accepted_dev [B, lmax] (-1 padded, root first), len_dev [B], next_token_dev [B] (the correction or
 * bonus token: emitted, not yet materialised), final_node_dev [B] (last accepted node, -1 = none):
 * the inputs of lumo_gdn_commit and of the next drafting step.  lmax >= tree depth.  Enqueues only. */
int lumo_tree_accept(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_accept_args* args, int lmax,
                     int32_t* accepted_dev, int32_t* len_dev, int32_t* next_token_dev,
                     int32_t* final_node_dev, void* stream);

/* ---- fused draft selection ------------------------------------------------------------------
 * Upstream of the tree (paper Sec. "Fuse draft selection without changing proposals"): from one
 * full-vocabulary logits row per drafting position, the spine token and three ordered sibling
 * candidates, written into caller-owned (graph-reusable) device buffers in one pass.
 *   spine[r]      = argmax_i logits[r, i], the lowest index among equal maxima;
 *   cand[r, 0..2] = the three largest entries, larger value first, among equal values the higher
 *                   index first (the paper states only that the two conventions differ; this is the
 *                   reading taken); duplicates of the spine token are kept.
 * logits: device [rows, V] contiguous, lumo_dtype f32 or bf16 (bf16 is widened exactly), no NaN
 * (entries of -inf are ordinary values).  rows >= 1, V >= 3.  split = CTAs that share one row:
 * 0 lets the library choose, else 1, 2, 4, 8 or 16; the result does not depend on it.  Enqueues
 * only; allocates nothing.  LUMO_ERR_ARG on bad sizes, dtype or split. */
typedef struct {
  int32_t rows, V;
  int32_t dtype;           /* lumo_dtype of logits */
  int32_t split;
  const void* logits;
} lumo_select_args;
int lumo_select_spine_top3(lumo_ctx* ctx, const lumo_select_args* args, int32_t* spine_dev /* [rows] */,
                           int32_t* cand_dev /* [rows, 3] */, void* stream);

/* ---- one GDN layer's tensors ----------------------------------------------------------- */
typedef struct {
  int32_t Hk, Hv, d;
  int32_t in_dtype;    /* lumo_dtype of x, conv_w, conv_b, conv_hist, q, k, v */
  int32_t gate_dtype;  /* lumo_dtype of alpha, beta */
  int32_t out_dtype;   /* lumo_dtype of out */
  float scale;         /* multiplies q (after normalisation); 1.0 = the paper's Eq. 3 */
  int32_t qk_l2norm;   /* 1: q <- q / sqrt(sum q^2 + l2_eps), same for k, inside the kernels */
  float l2_eps;
  int32_t n_state_rows; /* rows of the state / history pools (bounds check of state_row) */
  /* recorded operands: read by scan and commit; WRITTEN by verify when x != NULL */
  void* q;              /* [B, Ns, Hk, d] */
  void* k;              /* [B, Ns, Hk, d] */
  void* v;              /* [B, Ns, Hv, d] */
  const void* alpha;    /* [B, Ns, Hv] decay in (0, 1], post-activation (raw input if gate_mode = 1) */
  const void* beta;     /* [B, Ns, Hv] write strength in [0, 1], post-activation (raw input if gate_mode = 1) */
  /* convolution stage; x == NULL skips it in verify and skips the history update in commit */
  const void* x;        /* [B, Ns, C] raw projections, channels [q | k | v] */
  const void* conv_w;   /* [C, 4] tap 3 multiplies the node's own row */
  const void* conv_b;   /* [C] or NULL */
  void* conv_hist;      /* [rows, 3, C] committed raw inputs, oldest first; commit updates it */
  float* state;         /* [rows, Hv, d_v, d_k] fp32 pool; read-only in verify, updated by commit */
  const int32_t* state_row; /* [B] pool row of each sequence; -1 = skip the sequence */
  void* out;            /* [B, Ns, Hv, d_v] verify output */
  int32_t snapshot_mode;    /* 0 none, 1 list (snap_nodes), 2 every node */
  int32_t n_snap;           /* E: entries per sequence in snap_nodes (mode 1) / N (mode 2) */
  const int32_t* snap_nodes;/* [B, E] logical ids, -1 = unused (mode 1) */
  float* snap_out;          /* [B, E, Hv, d_v, d_k] fp32 node states */
  int32_t* status;          /* [B] lumo_seq_status, written by verify and by commit; may be NULL */
  /* Gate form.  0: alpha and beta hold post-activation values (above).  1: they hold the raw gate
   * inputs (Sec. "Sequential arithmetic and accepted-path replay": the verifier takes raw gate
   * inputs; the paper prints no formula, the reading taken is the Gated DeltaNet parametrisation)
   *   alpha = exp(-exp(a_log[h]) * softplus(alpha_in + dt_bias[h])),  beta = sigmoid(beta_in),
   * evaluated in fp32 inside verify and commit with the same code, so both see the same gates. */
  int32_t gate_mode;
  const float* a_log;       /* [Hv] fp32 (gate_mode 1) */
  const float* dt_bias;     /* [Hv] fp32 (gate_mode 1) */
} lumo_gdn_args;

/* Verifies all nodes of every tree through n_layers independent GDN layers (Algorithm 2,
 * "Verify paths; keep branch state temporary").  `layers` is a HOST array.  Read-only on
 * state and conv_hist.  All layers must share Hk, Hv, d and dtypes.  n_layers <= 64. */
int lumo_gdn_tree_verify(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_gdn_args* layers,
                         int n_layers, void* stream);

/* The tree scan for callers that must not allocate device memory.  (The paper has no counterpart:
 * this is a property of this library's scratch handling, not of the method.)
 *
 * lumo_gdn_tree_verify keeps the scan's state stack in memory that the context allocates the first
 * time a shape needs it.  Some callers cannot tolerate that: code running between the capture and
 * the replay of a CUDA graph's memory plan, a serving loop whose memory pool has already handed
 * every byte to the KV cache and the state banks, or a process whose allocator is owned by another
 * runtime.  This call runs the same scan kernel with the stack in a fixed array that is part of
 * the library image (lumo_static_stack_bytes() = 64 MiB, held by every GPU that loads the library
 * until the process exits).  It never calls cudaMalloc, cudaFree or any allocating routine.
 *
 *   - Runs the scan only, on the recorded operands q, k, v (the convolution stage needs no scratch;
 *     run it through lumo_gdn_tree_verify beforehand, or pass operands directly).  `x` is ignored.
 *   - Same arguments, outputs, snapshot modes and status words as lumo_gdn_tree_verify.
 *   - A shape whose persistent grid needs more stack than the array holds is refused with
 *     LUMO_ERR_UNSUPPORTED and a message that states both sizes; nothing is enqueued.
 *   - The first call on a device looks up the array's device address (once per device, with that
 *     device current).  Make that first call before starting any stream capture.
 *   - All calls share the one array.  Nothing in it has to start at zero (every stack level is
 *     written before it is read within a call), and it keeps the previous call's contents.  Two
 *     calls that overlap on the GPU (different streams, or graphs launched concurrently) race on
 *     it and corrupt each other's outputs: serialise them. */
int lumo_gdn_tree_scan_static(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_gdn_args* layers,
                              int n_layers, void* stream);
int64_t lumo_static_stack_bytes(void);

/* Diagnostic: how many entries of the visiting order one CTA of the tree convolution takes for this
 * tree batch, head shape and layer count on this context's device (16, 8 or 4; the three are separate
 * instantiations of the kernel, chosen so that the grid covers the GPU).  0 on a bad argument or a
 * host-only context.  Lets a parity test state which instantiation it exercised. */
int lumo_conv_rows_per_cta(const lumo_ctx* ctx, const lumo_tree_desc* desc, int Hk, int Hv, int d, int n_layers);

/* Replays accepted_dev [B, lmax] (logical ids, root first; entries at or beyond len_dev[b] are
 * ignored; 1 <= lmax <= 256, else LUMO_ERR_ARG and nothing is enqueued) from the pre-tree state with the recorded operands and publishes state and
 * convolution history in place (Algorithm 2, "Replay only the accepted path into native
 * recurrent state"; Algorithm 1, "Gather the convolution history for A into the native running
 * row").  len 0 leaves both bit-unchanged.  An invalid path sets status[b] and leaves the
 * sequence untouched.  Calling it twice advances twice. */
int lumo_gdn_commit(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_gdn_args* layers,
                    int n_layers, const int32_t* accepted_dev, const int32_t* len_dev, int lmax,
                    void* stream);

/* Commit of the previous cycle folded into this cycle's verify: the same result as
 *   lumo_gdn_commit(ctx, prev_desc, prev_layers, n_layers, accepted_dev, len_dev, lmax, stream);
 *   lumo_gdn_tree_verify(ctx, desc, layers, n_layers, stream);
 * with the running state read once: the scan replays the accepted path of the previous tree into
 * the state rows as it loads them, writes them back in place and verifies the new tree from there
 * (the paper's own design replays at once with a native update, Sec. "Sequential arithmetic and
 * accepted-path replay"; it names the fusion with the next verification as another system's choice,
 * Sec. "Temporary state versus recomputation").  prev_layers[l] and layers[l] must name the same
 * state, state_row and conv_hist and must share shapes, dtypes and options; the previous cycle's
 * q/k/v/x/gates must live in buffers of their own (they are read while the new ones are written).
 * prev_layers[l].status receives the commit's per-sequence status, layers[l].status the verify's.
 * The fused kernel serves d = 128, bf16 operands, trees of at most 64 nodes and depth 16,
 * lmax <= 16; every other case runs the two calls above one after the other.  Enqueues only. */
int lumo_gdn_commit_verify(lumo_ctx* ctx, const lumo_tree_desc* prev_desc, const lumo_gdn_args* prev_layers,
                           const int32_t* accepted_dev, const int32_t* len_dev, int lmax,
                           const lumo_tree_desc* desc, const lumo_gdn_args* layers, int n_layers, void* stream);

/* ---- attention half of the verifier ------------------------------------------------------
 * The hybrid model's full-attention layers see the same tree through the same slot map (Sec. "One
 * slot map governs attention and publication"; Sec. "State and the execution boundary": the
 * attention visibility relation selects the same logical prefix and ancestry as the recurrent path;
 * Algorithm 1, "Remap the accepted KV entries using the same logical-to-physical slot map").
 *
 * KV cache of one layer: k_cache, v_cache [n_cache_rows, max_positions, Hkv, dh] bf16 (or with the
 * head and position axes swapped, see kv_layout).  Sequence b
 * owns row cache_row[b]; positions [0, ctx_len[b]) hold the committed context, and the entry of tree
 * node i lives at position ctx_len[b] + slot[b][i] (the candidates occupy the physical suffix in slot
 * order; a spine-first slot map makes the principal chain contiguous there).  Queries and outputs
 * keep LOGICAL node order.  Node i attends to every context position and to the entries of its
 * ancestors and of itself; padding slots, other branches and anything beyond the suffix are never
 * read arithmetically (their bytes may be anything, NaN patterns included).  Query head h reads KV
 * head h / (Hq / Hkv).
 *
 * ctx_len and cache_row are DEVICE arrays [B] shared by all layers.  A sequence with
 * cache_row[b] outside [0, n_cache_rows) gets LUMO_SEQ_BAD_ROW, one with ctx_len[b] < 0 or
 * ctx_len[b] + Ns > max_positions LUMO_SEQ_BAD_CTX; such a sequence is skipped (write, publish) or
 * gets zero outputs and lse (attention).  Supported: dh = 128, Ns <= 256, 1 <= Hq / Hkv, n_layers <= 32.
 */
typedef struct {
  int32_t Hq, Hkv, dh;
  float scale;              /* logits = scale * q . k (the paper prints none: a parameter) */
  int32_t n_cache_rows, max_positions;
  void* k_cache;            /* [n_cache_rows, max_positions, Hkv, dh] bf16 */
  void* v_cache;
  const int32_t* ctx_len;   /* [B] */
  const int32_t* cache_row; /* [B] */
  const void* q;            /* [B, N, Hq, dh] bf16, logical node order (tree attention) */
  const void* k_new;        /* [B, N, Hkv, dh] bf16, logical node order (write) */
  const void* v_new;
  float* out;               /* [B, N, Hq, dh] fp32 (tree attention) */
  float* lse;               /* [B, N, Hq] fp32 natural-log sum of exp of the logits; may be NULL */
  int32_t kv_layout;        /* 0: caches are [n_cache_rows, max_positions, Hkv, dh] (a position's heads adjacent);
                               1: [n_cache_rows, Hkv, max_positions, dh] (a head's positions adjacent: a tile of keys is
                               one contiguous 32 KB run, which the attention kernel reads at a higher HBM efficiency) */
  int32_t n_splits;         /* partitions of the key range per (sequence, KV head, row tile): 0 = the key tiles of the
                               whole call are dealt out evenly over the SMs (a unit is cut wherever a share ends),
                               else 1..32 equal partitions (Sec. "Evaluation Setup": the paper's deployment used 4) */
  int32_t* status;          /* [B] lumo_seq_status; may be NULL */
} lumo_attn_args;

/* Writes the tree's keys and values through the slot map: entry of node i of sequence b goes to
 * position ctx_len[b] + slot[b][i] of row cache_row[b] (Sec. "One slot map governs attention and
 * publication": the same permutation is applied to KV write slots and to the mask's key columns).
 * A pure scatter, bit-exact.  `layers` is a HOST array; all layers share shapes, ctx_len and cache_row. */
int lumo_kv_write_tree(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_attn_args* layers, int n_layers,
                       void* stream);

/* Ancestry-masked decode attention of every tree node over [context ; tree entries]:
 *   out[b,i,h,:] = sum_p softmax_p(scale q[b,i,h] . k[p]) v[p],  p over the visible positions,
 * on tcgen05 tensor cores: the query rows of all heads that share a KV head form one 128-row tile
 * (rows = (h mod G) * N + i, G = Hq / Hkv; further tiles when G N > 128), so a staged key/value tile
 * is read once for the whole group (Sec. "One slot map governs attention and publication": grouped
 * query heads share staged KV tiles); the key range of a unit is cut into partitions handled by
 * different CTAs, combined in key order by the log-sum-exp rule (same section: split-K context
 * partitions).  Probabilities enter the second product rounded to bf16; all sums are fp32.
 * The result is bitwise reproducible for a given device, shape and n_splits; other partitionings differ
 * by rounding.
 * Needs max_positions * Hkv * dh * 2 bytes < 2^40 per cache row.  Enqueues only; library scratch for
 * the partial results grows on the first call with a shape.  All attention calls of a context share that
 * scratch: enqueue them on one stream (or otherwise serialise them).  After one call with a shape the call
 * allocates nothing and can be captured into a CUDA graph.  If a bounded device-side wait runs
 * out, every sequence of the call gets LUMO_SEQ_TIMEOUT and the outputs of the call are invalid. */
int lumo_tree_attention(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_attn_args* layers, int n_layers,
                        void* stream);

/* Publication of the accepted path in the KV cache (Algorithm 1, "remap KV"): for t < len[b] the entry
 * at ctx_len[b] + slot[b][accepted[b][t]] moves to position ctx_len[b] + t, all reads before any write;
 * entries already in place move no bytes (a spine-first slot map makes publication of the principal
 * chain free).  ctx_len_out[b] = ctx_len[b] + len[b] (ctx_len_out may be NULL; it must not alias
 * ctx_len).  Same path rules, lmax bound and status codes as lumo_gdn_commit; an invalid path leaves
 * the row untouched and ctx_len_out[b] = ctx_len[b].  Bit-exact. */
int lumo_kv_publish(lumo_ctx* ctx, const lumo_tree_desc* desc, const lumo_attn_args* layers, int n_layers,
                    const int32_t* accepted_dev, const int32_t* len_dev, int lmax, int32_t* ctx_len_out,
                    void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LUMO_GDN_H_ */
