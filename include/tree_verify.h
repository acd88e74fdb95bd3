/*
 * tree_verify.h -- C ABI of the tree-verification library for recurrent
 * linear-attention layers (gated linear attention and the gated delta rule).
 *
 * What it computes.  A hybrid model keeps, per request, layer and state head,
 * one committed state S_pre.  A drafter proposes a token tree of T nodes with
 * parent map pi (nodes indexed parent before child; pi(i) = -1 marks a child
 * of the virtual root whose state is S_pre).  Every node i carries
 * q_i, k_i (dk), v_i (dv), a decay gate alpha_i > 0 (the paper's gamma_i) and,
 * for the delta rule, a write gate beta_i.  Sequential execution along a
 * root-to-node path applies (Section II-B Eq. 1; Section IV-A Table II,
 * "Sequential rule")
 *
 *     S~_i = alpha_i S_pi(i),   u_i = beta_i (v_i - S~_i^T k_i)   [delta]
 *                               u_i = v_i                         [gated]
 *     S_i  = S~_i + k_i u_i^T,  o_i = S_i^T q_i.
 *
 * tv_tree_verify returns o_i (and optionally u_i) for ALL nodes in one pass
 * from the single immutable S_pre, without forming any per-node state
 * (Section IV-A Theorem 1, Eq. 2, with Lemmas 1-3).  tv_commit_path then
 * writes the one state that must persist, the state at the end of the accepted
 * root-to-node path (Section IV-D Eq. 10).
 *
 * Memory layout (dense, row-major, innermost index last, unless tv_dims carries
 * strides for the node-indexed tensors -- see tv_strides):
 *     S_pre, S_new : float  [L][B][H][dv][dk]   (the serving cache layout
 *                    "[H, dv, dk]" of Section IV-D, i.e. the transpose of the
 *                    paper's S in R^{dk x dv})
 *     q, k         : float or bf16 [L][B][H][T][dk]   ([L][B][Hk][T][dk] with
 *                    grouped key heads, see tv_dims.Hk)
 *     v            : float or bf16 [L][B][H][T][dv]
 *     alpha, beta  : float  [L][B][H][T]
 *     O, U         : float  [L][B][H][T][dv]
 * L = number of recurrent layers handled by one call (independent problems
 * that share the trees and the accepted nodes).  Pointers marked "dev" are
 * device pointers on the current CUDA device, 16-byte aligned; "host" are
 * ordinary host pointers.  The caller owns every tensor and the stream; the
 * library owns tv_tree objects only.
 *
 * Every function returns TV_OK (0) or a negative tv_status.  Nothing throws,
 * aborts or prints.  Arguments are validated on the host before any launch.
 * Preconditions that cannot be checked on the host: all inputs finite,
 * alpha > 0.
 */
#ifndef TREE_VERIFY_H_
#define TREE_VERIFY_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TV_MAX_NODES 128   /* T <= 128: ancestor sets are 128-bit masks   */
#define TV_MAX_DIM   128   /* dk, dv <= 128, multiples of 4               */
#define TV_STATIC_MAX_TREES 128  /* capacity of tv_tree_verify_static       */

typedef enum tv_status {
  TV_OK = 0,
  TV_ERR_BAD_ARG = -1,        /* null / misaligned pointer, size out of range   */
  TV_ERR_INVALID_TREE = -2,   /* parent[i] >= i or parent[i] < -1               */
  TV_ERR_UNSUPPORTED = -3,    /* shape outside what the kernels cover           */
  TV_ERR_CUDA = -4,           /* a CUDA runtime call failed (tv_last_cuda_error)*/
  TV_ERR_NOT_UPLOADED = -5,   /* tree metadata not on the device yet            */
  TV_ERR_DEVICE_TIMEOUT = -6, /* a bounded device-side wait ran out             */
  TV_ERR_NOMEM = -7,
  TV_ERR_TOO_LARGE = -8       /* size beyond a fixed, documented capacity       */
} tv_status;

enum { TV_GATED = 0, TV_GATED_DELTA = 1 };  /* update rule                      */
enum { TV_F32 = 0, TV_BF16 = 1 };           /* dtype of q, k, v                 */
enum { TV_IMPL_AUTO = 0, TV_IMPL_SIMT = 1, TV_IMPL_TC = 2 }; /* kernel choice   */

typedef struct tv_tree tv_tree;             /* opaque, library-owned            */

/* Element strides of a node-indexed tensor (d contiguous): element (layer l, request b,
 * head h, node t, channel c) sits at (l * B + b) * b + h * h + t * t + c.  All three zero
 * means the dense head-major layout of the table above.  Token-major projections
 * [B][T][H][d] are {T*H*d, d, H*d}; q, k and v taken in place from one fused projection
 * [B][T][C] are three base pointers with {T*C, d, C}.  Strides are multiples of 16 bytes
 * for q, k, v, O, U (any value for alpha, beta) and must not make elements overlap.
 * (Section IV-C folds "layout conversion" into the stages: this is that, with no copy.)   */
typedef struct tv_strides {
  int64_t b, h, t;
} tv_strides;

typedef struct tv_dims {
  int32_t L, B, H, T, dk, dv;
  int32_t rule;        /* TV_GATED / TV_GATED_DELTA                             */
  int32_t qkv_dtype;   /* TV_F32 / TV_BF16                                      */
  int32_t impl;        /* TV_IMPL_AUTO picks a tensor-core kernel when the
                          shape allows it (bf16, dk = dv = 128; gated rule
                          also dk = dv = 64 in dense layouts; delta rule: tree
                          depth <= 15) and the SIMT fp32 kernel otherwise;
                          TV_IMPL_TC returns TV_ERR_UNSUPPORTED instead of
                          falling back                                          */
  int32_t Hk;          /* grouped key heads (Section IV-D: a K factor shared by
                          several state heads is stored once): q and k have Hk
                          heads, [L][B][Hk][T][dk], and state head h reads
                          q/k head h / (H / Hk).  0 means Hk = H; H % Hk == 0. */
  tv_strides qk;       /* layout of q and k (heads = Hk)                        */
  tv_strides v;        /* layout of v                                           */
  tv_strides gate;     /* layout of alpha and beta (d = 1)                      */
  tv_strides out;      /* layout of O and U                                     */
                       /* Strided layouts are for dense trees; a packed forest
                          (tv_forest_build) keeps its planes and returns
                          TV_ERR_UNSUPPORTED when any stride is set.            */
} tv_dims;

const char* tv_strerror(int status);
int tv_version(void);
/* cudaError_t value of the last failed CUDA call on this thread (0 if none). */
int tv_last_cuda_error(void);

/* ---- tree metadata (Section IV-A Table II: Anc(i), d, M^-; Section IV-C
 * "Round-level topology preprocessing": built once per request and round,
 * reused by every layer and head, in fixed buffers) -------------------------
 *
 * tv_tree_build: host only, no CUDA call.  parent is host int32
 * [n_trees][n], -1 <= parent[t][i] < i, 1 <= n <= TV_MAX_NODES.  Produces, per
 * node, the strict-ancestor set as a 128-bit mask (bit j&63 of word j>>6 set
 * iff j in Anc(i): row i of M^-), depth[i] = |Anc(i)| (0 for a root child) and
 * per tree max_depth = d.  *out is owned by the library until tv_tree_free.
 * Returns TV_ERR_INVALID_TREE (and leaves *out NULL) for a malformed parent
 * array.                                                                      */
int tv_tree_build(const int32_t* parent /*host*/, int32_t n_trees, int32_t n,
                  tv_tree** out);
/* Same sizes, new topology, no allocation (fixed buffers across rounds).      */
int tv_tree_rebuild(tv_tree* tree, const int32_t* parent /*host*/);
/* Copy metadata out (host): anc [n_trees][n][2], depth [n_trees][n],
 * max_depth [n_trees].  Any output pointer may be NULL.                       */
int tv_tree_meta(const tv_tree* tree, uint64_t* anc, int32_t* depth,
                 int32_t* max_depth);
/* n_trees, n and the maximum depth over all trees.                            */
int tv_tree_info(const tv_tree* tree, int32_t* n_trees, int32_t* n,
                 int32_t* max_depth_all);
/* Accepted-path indices (Section IV-D: P(a) = Anc(a) + {a}, topological
 * order).  accepted is host int32 [n_req]; request r uses tree r (tree 0 when
 * n_trees == 1); accepted[r] = -1 means no draft token accepted (len 0).
 * path is host int32 [n_req][path_stride], path_stride >= max_depth_all + 1,
 * unused entries set to -1; len is host int32 [n_req].                        */
int tv_tree_path(const tv_tree* tree, const int32_t* accepted, int32_t n_req,
                 int32_t* path, int32_t path_stride, int32_t* len);
/* Put the metadata on the current device, on `stream` (a cudaStream_t): one
 * small kernel derives the same masks and depths on the device from the parent
 * arrays (Section IV-C: once per request and round, fixed buffers).  Tree sets
 * of up to 16384 nodes travel in that kernel's parameters; larger ones are
 * staged in pinned host memory that the kernel reads.  The first call allocates
 * the device mirror and the staging block; later calls (after tv_tree_rebuild)
 * allocate nothing.  Asynchronous; kernels launched
 * later on the same stream see the result.                                     */
int tv_tree_upload(tv_tree* tree, void* stream);
/* Copy the DEVICE-built masks and depths back to host arrays (same shapes as
 * tv_tree_meta) and synchronise `stream`: lets a caller check them bit for bit
 * against tv_tree_meta.                                                       */
int tv_tree_meta_device(tv_tree* tree, uint64_t* anc, int32_t* depth, void* stream);
/* Synchronises `stream` and reports whether any kernel launched with this tree
 * since its last upload gave up on a bounded device-side wait (a TMA or tensor-
 * core completion that never came): TV_OK or TV_ERR_DEVICE_TIMEOUT.  After a
 * timeout the outputs of that launch are undefined; the context stays usable.
 * TV_ERR_UNSUPPORTED: the trees of the last tv_forest_upload_device were deeper
 * than the bound that call was given.  TV_ERR_CUDA: a tensor-core kernel (or
 * tv_tree_conv, whose row boxes arrive by TMA) found its shared-memory window
 * off the boundary its tiles need and left without computing (outputs
 * undefined, as after a timeout).                                             */
int tv_tree_device_status(tv_tree* tree, void* stream);
/* Self-test of that mechanism: launches one CTA that waits, with a limit of a
 * few milliseconds, on a barrier nothing ever signals, and writes what the
 * kernels would report (TV_ERR_DEVICE_TIMEOUT) to the DEVICE int32 *status.
 * Nothing faults or hangs; the context stays usable.                          */
int tv_selftest_wait_timeout(int32_t* status /*dev*/, void* stream);
int tv_tree_free(tv_tree* tree);

/* ---- packed forest (Section V-B "CUDA Graph-native packed-forest execution":
 * variable-sized trees packed topologically into one flat-ragged forest of
 * fixed total capacity, described by request offsets, parent indices and
 * compact ancestor metadata; only tiles internal to a request are computed) ---
 *
 * tv_forest_build: host only.  Request r owns nodes offsets[r] .. offsets[r+1]-1
 * of the flat forest (offsets host int32 [n_req+1], offsets[0] = 0, between 1
 * and n_max <= TV_MAX_NODES nodes each, offsets[n_req] <= capacity);
 * parent_flat (host int32 [offsets[n_req]]) holds each node's parent as an
 * index LOCAL to its request, -1 <= parent < local index.  The handle is used
 * with the same calls as a dense one (upload, verify, commit, conv), with
 * tv_dims.T = n_max and B = n_req, but the node-indexed tensors are packed
 * planes of `capacity` rows:
 *     q, k        [L][Hk][capacity][dk]      v, O, U  [L][H][capacity][dv]
 *     alpha, beta [L][H][capacity]           (row offsets[r] + i = node i of r)
 * S_pre / S_new keep [L][B][H][dv][dk]; accepted[r] is local to request r.
 * Rows at and beyond offsets[n_req] are never read or written.  Metadata
 * (tv_tree_meta, tv_tree_meta_device) stays padded per request: n_max entries
 * each, padding entries have empty ancestor sets.  tv_tree_path works as for
 * dense trees.  tv_forest_rebuild: new topology and offsets, same n_req, n_max
 * and capacity, no allocation (fixed buffers across rounds).
 * Errors: TV_ERR_BAD_ARG (offsets not increasing from 0, a request with no or
 * more than n_max nodes), TV_ERR_TOO_LARGE (more nodes than capacity),
 * TV_ERR_INVALID_TREE.                                                        */
int tv_forest_build(const int32_t* parent_flat /*host*/, const int32_t* offsets /*host*/,
                    int32_t n_req, int32_t n_max, int32_t capacity, tv_tree** out);
int tv_forest_rebuild(tv_tree* forest, const int32_t* parent_flat /*host*/,
                      const int32_t* offsets /*host*/);

/* ---- batch-wide utility allocation (Section V-A "Batch-wide utility
 * allocation") and device-side forest materialisation (Section V-B) ----------
 * Every request brings a candidate tree of n_cand <= TV_MAX_NODES nodes (node 0
 * = the tree's root, parent -1; -1 <= parent[i] < i) and the drafter's
 * conditional probability p_draft of every node, 0 <= p <= 1.  tv_budget_select
 * scores node v by rho(v) = rho(parent(v)) * p_draft(v) (float32, one rounding
 * per edge; rho of a root child is its own p), keeps the root of every tree
 * and, of all other nodes of the batch, the budget - n_req highest rho (ties:
 * lower (request, node) index first), and packs the kept nodes request by
 * request in their original order:
 *   rho           float [n_req][n_cand]
 *   counts        int32 [n_req]     kept nodes per request (the budget q_r)
 *   offsets       int32 [n_req+1]   prefix sums of counts
 *   parent_packed int32 [n_req][n_cand]  parents renumbered locally, padded with -1
 *   node_id       int32 [budget]    r * n_cand + i of every packed row, -1 past the forest
 * All pointers are DEVICE pointers (4-byte aligned; workspace 16-byte aligned,
 * tv_budget_workspace_bytes(n_req, n_cand) bytes); nothing is allocated and the
 * host is not synchronised.  *status (device int32, may be NULL) receives
 * TV_ERR_INVALID_TREE if a parent is out of range (it is then treated as -1).
 * n_req <= 1024, n_req <= budget.  parent_packed and offsets are exactly what
 * tv_forest_upload_device reads: it derives the masks and depths of a forest
 * handle (tv_forest_build with the same n_req, n_max = n_cand, capacity >=
 * budget) from DEVICE memory, with no host copy.  max_depth_bound must bound the
 * depth of every candidate tree (the kernel choice depends on it).  The device
 * checks it: a node with more ancestors keeps only its nearest max_depth_bound
 * of them, so every kernel stays within its tables, the results of that round
 * are not the tree's, and tv_tree_device_status returns TV_ERR_UNSUPPORTED
 * until the next upload.  After it the handle's host-side metadata is stale:
 * tv_tree_meta and tv_tree_path return TV_ERR_UNSUPPORTED until the next
 * tv_forest_rebuild + tv_tree_upload.                                          */
size_t tv_budget_workspace_bytes(int32_t n_req, int32_t n_cand);
int tv_budget_select(const int32_t* parent /*dev*/, const float* p_draft /*dev*/, int32_t n_req,
                     int32_t n_cand, int32_t budget, float* rho, int32_t* counts, int32_t* offsets,
                     int32_t* parent_packed, int32_t* node_id, void* workspace, int32_t* status,
                     void* stream);
int tv_forest_upload_device(tv_tree* forest, const int32_t* parent_padded /*dev*/,
                            const int32_t* offsets /*dev*/, int32_t max_depth_bound, void* stream);

/* ---- verification (Section IV-A Theorem 1, Eq. 2; Eq. 4; Lemma 2 Eq. 5) ----
 *
 * For every layer, request, head and node i:
 *     O[i] = P_i S_pre^T q_i + sum_{j in Anc(i)+{i}} (P_i/P_j)(q_i.k_j) u_j,
 * P_i = prod of alpha over Anc(i)+{i}; u_j = v_j (TV_GATED) or the solution of
 * the ancestor-masked system (I+G)U = R of Lemma 2 (TV_GATED_DELTA).
 * tree must hold 1 tree (shared by the batch) or B trees, with n == T, and be
 * uploaded.  S_pre is read only.  beta may be NULL for TV_GATED.  U may be
 * NULL; when given it receives the correction rows u_i (for TV_GATED a copy of
 * v widened to float).  One asynchronous launch sequence on `stream`; no
 * allocation, no host synchronisation.  Stream order: the kernel may be
 * scheduled while the library kernel directly in front of it on the stream
 * drains (a tree upload, another tv_tree_verify, tv_tree_conv), and asks for
 * its first S_pre tile then; everything else it reads after that kernel has
 * completed.  None of those kernels writes a state, and behind any other work
 * (tv_commit_path included) the kernel starts after that work, as usual -- a
 * caller's own kernel that writes S_pre and releases its dependents early
 * (programmatic dependent launch) is the one thing that must not sit directly
 * in front of this call.                                                      */
int tv_tree_verify(const tv_tree* tree, const tv_dims* dims,
                   const float* S_pre /*dev*/,
                   const void* q /*dev*/, const void* k /*dev*/, const void* v /*dev*/,
                   const float* alpha /*dev*/, const float* beta /*dev or NULL*/,
                   float* O /*dev*/, float* U /*dev or NULL*/,
                   void* stream);

/* ---- verification without any allocation ------------------------------------
 * (The paper has no counterpart: this entry exists for this library's users.)
 *
 * Some callers may not allocate device or pinned memory at all: code inside a
 * CUDA-graph capture, a serving loop whose memory was carved up at start-up,
 * a plug-in in a process that owns the allocator, or a latency-critical path
 * that cannot afford the implicit synchronisation of an allocation.  The
 * regular path allocates in tv_tree_build and in the first tv_tree_upload.
 * This call does the same verification as tv_tree_verify but takes the parent
 * arrays straight from DEVICE memory (int32 [n_trees][T], n_trees = 1 or B, as
 * a drafter running on the GPU leaves them) and keeps the derived masks and
 * depths in a fixed array inside the library's device image: 384 KiB that
 * every GPU which loads the library holds until the process exits.  It calls
 * no cudaMalloc/cudaFree and no allocating library routine.
 *
 * Limits: n_trees <= TV_STATIC_MAX_TREES and T <= TV_MAX_NODES, otherwise
 * TV_ERR_TOO_LARGE / TV_ERR_UNSUPPORTED is returned and nothing is launched.
 * The delta rule runs on the general fp32 kernel here (the tree depth is not
 * known on the host).
 * The first call on each device looks up the device address of that array
 * (with that device current); make that first call outside any stream capture.
 * All calls share the array and it keeps the last call's metadata (the part a
 * call needs is rewritten, and its status word cleared, by the call itself):
 * two calls whose kernels may overlap on the GPU -- different streams without
 * ordering -- race on it; calls on one stream are safe.
 * The parents cannot be validated on the host: a parent outside [-1, i) is
 * treated as -1 and TV_ERR_INVALID_TREE is written to *status; a device-side
 * wait that ran out writes TV_ERR_DEVICE_TIMEOUT.  status is a DEVICE int32
 * that the caller zeroes beforehand, or NULL.                                 */
int tv_tree_verify_static(const int32_t* parent /*dev*/, int32_t n_trees, const tv_dims* dims,
                          const float* S_pre /*dev*/,
                          const void* q /*dev*/, const void* k /*dev*/, const void* v /*dev*/,
                          const float* alpha /*dev*/, const float* beta /*dev or NULL*/,
                          float* O /*dev*/, float* U /*dev or NULL*/,
                          int32_t* status /*dev or NULL*/, void* stream);

/* ---- accepted-path commit (Section IV-D Eq. 10; Lemma 1 Eq. 3) -------------
 *
 *     S_new = P_a S_pre + sum_{j in P(a)} (P_a/P_j) k_j u_j^T   (stored [dv][dk])
 * for the accepted terminal node a = accepted[b] of each request, all L layers
 * and all heads in one launch.  accepted is a DEVICE int32 [B] (it comes from
 * the sampler), each value in [-1, T); -1 leaves the slot unchanged (nothing
 * is read or written when S_new == S_pre, S_pre is copied otherwise).  Values
 * outside [-1, T) are treated as -1.  U: the corrections written by
 * tv_tree_verify, or NULL -- then TV_GATED uses u_j = v_j and TV_GATED_DELTA
 * re-derives u_j along the accepted path from S_pre (needs dk in {64,128}).
 * S_new may alias S_pre exactly (in place) or not overlap it at all.
 * Stream order: when the call directly follows tv_tree_verify, tv_tree_upload,
 * tv_forest_upload_device or tv_tree_conv on the same stream, the commit grid
 * may be scheduled while that kernel drains and read S_pre and accepted early;
 * it reads the tree metadata and U, and writes S_new, only after that kernel
 * has completed -- and that kernel lets it start only once everything in front
 * of itself has completed.  (Behind any other work it starts after that work,
 * as usual.)  So accepted and S_pre must not be outputs of the library call
 * directly in front of it -- U and the tree metadata are the only ones that
 * may be.                                                                     */
int tv_commit_path(const tv_tree* tree, const tv_dims* dims,
                   const int32_t* accepted /*dev [B]*/,
                   const float* S_pre /*dev*/,
                   const void* k /*dev*/, const void* v /*dev*/,
                   const float* alpha /*dev*/, const float* beta /*dev or NULL*/,
                   const float* U /*dev or NULL*/,
                   float* S_new /*dev*/,
                   void* stream);

/* The same commit for a model whose recurrent layers own their caches separately
 * (Section IV-D: "all linear layers" are committed together; Section V-B "Unified
 * cross-layer state commit": one batched launch from per-request path descriptors
 * shared by all layers).  Every table is a HOST array of n_layers DEVICE pointers,
 * one tensor of a single layer each, in the layouts and with the alignment of
 * tv_commit_path (dims->L is ignored; dims' strides apply inside every layer).
 * v, beta, U may be NULL as tables under the rules of tv_commit_path.  The
 * pointers travel in the kernel's parameters: ONE launch for up to 64 layers (one
 * more per further 64), no device-side table to keep alive, no allocation.
 * S_new[l] == S_pre[l] for every layer (in place) or for none; otherwise no
 * S_new[l] may overlap any S_pre[m].  Stream order as for tv_commit_path.       */
int tv_commit_path_layers(const tv_tree* tree, const tv_dims* dims,
                          const int32_t* accepted /*dev [B]*/, int32_t n_layers,
                          const float* const* S_pre /*host [n_layers] of dev*/,
                          const void* const* k, const void* const* v,
                          const float* const* alpha, const float* const* beta,
                          const float* const* U, float* const* S_new,
                          void* stream);

/* ---- host-buffer round ------------------------------------------------------
 * The whole hot path (tv_tree_build -> tv_tree_verify -> tv_commit_path, i.e.
 * Section IV-C topology step, Theorem 1 and Eq. 10 in sequence) for callers
 * whose tensors live in HOST memory (pinned memory makes the copies
 * asynchronous).  A session owns device copies sized for `dims` (allocated
 * once by tv_session_create on the current device; n_trees is 1 or B).
 * tv_session_round copies parent/accepted/S_pre/q/k/v/alpha/beta to the device,
 * verifies, commits in place on the device copy (the delta rule commits from
 * the corrections U that verify wrote), copies O and S_new back and
 * synchronises before returning.  The requests are handled in up to eight
 * groups that flow through three streams of the session's own -- copies in,
 * kernels, copies out, chained by events per group; all ordered after the work
 * already queued on `stream`, and `stream` waits for them -- so that the
 * copies in, the kernels and the copies out of different groups overlap.  All pointers are
 * host pointers in the layouts above; beta may be NULL for TV_GATED.           */
typedef struct tv_session tv_session;
int tv_session_create(const tv_dims* dims, int32_t n_trees, tv_session** out);
int tv_session_round(tv_session* s, const int32_t* parent /*[n_trees][T]*/,
                     const int32_t* accepted /*[B]*/, const float* S_pre,
                     const void* q, const void* k, const void* v,
                     const float* alpha, const float* beta,
                     float* O, float* S_new, void* stream);
int tv_session_free(tv_session* s);

/* ---- Stage 1: tree-parallel convolution and gate preparation (Section II-A,
 * Section IV-C "Stage 1") -----------------------------------------------------
 * The layer's front end: a short causal depthwise convolution whose taps for a
 * tree node are the node itself and its nearest ancestors along the
 * root-to-node path, continued into the committed context once the path ends,
 * followed by bias and SiLU.  One layer per call.  With C = H*(2*dk+dv) and the
 * channel order [q heads | k heads | v heads] (head-major inside each block):
 *
 *   y[b][i][c] = SiLU( bias[c] + sum_{r<W} weight[c][W-1-r] * in_r(b,i)[c] ),
 *   in_0 = x[b][i], in_1 = x[b][pi(i)], ...; past the root: ctx[b][W-2],
 *   ctx[b][W-3], ...                          SiLU(z) = z / (1 + exp(-z))
 *
 * and y is written head-major, in the layout tv_tree_verify reads:
 *   q, k [B][H][T][dk], v [B][H][T][dv].  normalize_qk != 0 divides every q and
 *   k head vector by sqrt(sum of squares + eps) (the paper folds
 *   "normalisation" into its stages without a formula; this is the reading).
 * Gate preparation (optional: pass gate_a == NULL to skip).  The paper names the
 * step only; the formulas are those of the Gated DeltaNet layer it cites:
 *   alpha[b][h][i] = exp(-exp(A_log[h]) * softplus(gate_a[b][i][h] + dt_bias[h]))
 *   beta [b][h][i] = 1 / (1 + exp(-gate_b[b][i][h]))      (gate_b may be NULL)
 *
 * Device pointers, all owned by the caller, none retained:
 *   x      [B][T][C]   io_dtype        ctx    [B][W-1][C] io_dtype, oldest row first
 *   weight [C][W]      float           bias   [C] float or NULL
 *   gate_a, gate_b [B][T][H] io_dtype  A_log, dt_bias [H] float
 *   q, k, v            io_dtype        alpha, beta [B][H][T] float
 * x, ctx, weight, bias, q, k, v 16-byte aligned; dk, dv multiples of 8 (bf16) or 4 (float),
 * at most 256; 1 <= W <= TV_CONV_MAX_TAPS; T <= TV_MAX_NODES.  The tree must be
 * uploaded (1 tree shared by all requests, or B trees).  With a packed forest
 * (tv_forest_build; T = n_max, B = n_req) the node-indexed tensors are packed
 * like those of tv_tree_verify: x [capacity][C], gate_a, gate_b [capacity][H]
 * (row offsets[r] + i = node i of request r), q, k, v [H][capacity][d],
 * alpha, beta [H][capacity]; ctx keeps [B][W-1][C].  Outputs must not alias
 * inputs.  Asynchronous on `stream`; returns a tv_status, launches nothing on
 * an error.  The kernel's waits (row boxes arriving by TMA) are bounded like
 * those of the tensor-core kernels: tv_tree_device_status(tree) reports one
 * that ran out. */
#define TV_CONV_MAX_TAPS 8
typedef struct tv_conv_dims {
  int32_t B, H, T, dk, dv;
  int32_t W;             /* taps, including the current token           */
  int32_t io_dtype;      /* tv_dtype of x, ctx, gate_a, gate_b, q, k, v  */
  int32_t normalize_qk;  /* 0 / 1                                        */
  float eps;             /* added under the square root                  */
  int32_t impl;          /* TV_IMPL_AUTO / TV_IMPL_SIMT: the CUDA-core kernel (the only
                            one); TV_IMPL_TC returns TV_ERR_UNSUPPORTED      */
} tv_conv_dims;

int tv_tree_conv(const tv_tree* tree, const tv_conv_dims* dims, const void* x, const void* ctx,
                 const float* weight, const float* bias, const void* gate_a, const void* gate_b,
                 const float* A_log, const float* dt_bias, void* q, void* k, void* v,
                 float* alpha, float* beta, void* stream);

/* The convolution's context after the accepted path is committed (the
 * counterpart, for the front end, of Section IV-D's state commit; implied, not
 * spelled out, by the paper): ctx_new[b] = the last W-1 rows of
 * [ctx[b] rows, x[b] along the accepted root-to-node path].  accepted[b] = -1
 * keeps ctx[b].  accepted [B] int32 (device), ctx_new [B][W-1][C] io_dtype;
 * ctx_new == ctx (in place) is allowed, partial overlap is not. */
int tv_conv_commit(const tv_tree* tree, const tv_conv_dims* dims, const int32_t* accepted,
                   const void* x, const void* ctx, void* ctx_new, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TREE_VERIFY_H_ */
