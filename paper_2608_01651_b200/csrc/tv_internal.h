// Internal declarations shared by the translation units of libtreeverify.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "tree_verify.h"

struct tv_tree {
  int32_t n_trees = 0, n = 0, max_depth_all = 0;
  // host metadata
  std::vector<int32_t> parent, depth, max_depth;
  std::vector<uint64_t> anc;  // [n_trees][n][2]
  // device mirror: one blob = anc | depth | parent, staged through pinned memory
  int device = -1;
  void* d_blob = nullptr;
  void* h_stage = nullptr;
  size_t blob_bytes = 0;
  const uint64_t* d_anc = nullptr;
  const int32_t* d_depth = nullptr;
  const int32_t* d_parent = nullptr;
  uint64_t* d_anc_w = nullptr;
  int32_t* d_depth_w = nullptr;
  int32_t* d_parent_w = nullptr;
  int32_t* d_status = nullptr;  // device status: [0] timeout flag (0 = ok), cleared by every upload;
                                // [1] generation of the last upload whose trees broke their depth bound
  int32_t upload_gen = 0;       // generation of the latest upload (counts from 1)
  bool uploaded = false;
  bool host_meta_valid = true;   // false after tv_forest_upload_device: the topology lives on the device only
  // Packed forest (tv_forest_build): tree t has offsets[t+1] - offsets[t] <= n real nodes (its
  // metadata slab is padded to n with root children) and its tensor rows start at offsets[t] in
  // every (layer, head) plane of `capacity` rows.  Empty for a dense tree set.
  std::vector<int32_t> offsets;
  int32_t capacity = 0;
  const int32_t* d_offsets = nullptr;
  int32_t* d_offsets_w = nullptr;
  cudaEvent_t staged[2] = {nullptr, nullptr};  // the device has read staging slot 0 / 1
  const int32_t* h_stage_dev = nullptr;          // device view of the pinned staging block
  int stage_slot = 0;
};

// Kernel-side view of the tree metadata.
struct TreeDev {
  const uint64_t* anc;    // [n_trees][T][2]
  const int32_t* depth;   // [n_trees][T]
  const int32_t* parent;  // [n_trees][T]
  int32_t n_trees;
  int32_t max_depth_all;
  const int32_t* offsets;  // packed forest: [n_trees + 1] first tensor row of each tree; else null
  int32_t capacity;        // packed forest: rows of one (layer, head) plane
};

// Element strides of a node-indexed tensor: element (layer l, request b, head h, node t, channel c)
// sits at (l * B + b) * b + h * h + t * t + c.  Always resolved (never all zero) by the time a
// launcher sees them; a packed forest ignores them (its planes are addressed by request offsets).
struct Str3 {
  int64_t b, h, t;
};
struct Layout {
  Str3 qk, v, gate, out;   // q and k | v | alpha and beta | O and U
};
// Fills `out` from the caller's tv_dims (zero strides = dense head-major) and validates it.
int tv_resolve_layout(const tv_dims* d, bool packed, Layout* out);

struct VerifyArgs {
  TreeDev tree;
  int32_t L, B, H, T, dk, dv, rule, bf16;
  int32_t Hk;  // q/k heads (H % Hk == 0); state head h reads q/k head h / (H / Hk)
  Layout lay;
  const float* S_pre;
  const void* q;
  const void* k;
  const void* v;
  const float* alpha;
  const float* beta;
  float* O;
  float* U;
};

// Commit: dimensions and flags; the tensors come layer by layer from a CommitLayers table, so that
// layers that own their caches separately are committed by the same single launch as layers
// stacked in one allocation.  Node-indexed tensors are addressed within their layer (the layer
// index of Layout's (l * B + b) is always 0 here).
struct CommitArgs {
  TreeDev tree;
  int32_t L, B, H, T, dk, dv, rule, bf16;   // L = layers of this launch (<= kCommitMaxLayers)
  int32_t Hk;
  int32_t has_U;      // corrections given (else v, or the delta rule re-derived along the path)
  int32_t in_place;   // every layer's S_new is its S_pre
  Layout lay;
  const int32_t* accepted;
};
constexpr int kCommitMaxLayers = 64;
struct CommitLayers {
  const float* S_pre[kCommitMaxLayers];
  float* S_new[kCommitMaxLayers];
  const void* k[kCommitMaxLayers];
  const void* v[kCommitMaxLayers];
  const float* alpha[kCommitMaxLayers];
  const float* beta[kCommitMaxLayers];
  const float* U[kCommitMaxLayers];
};

// True when every node-indexed tensor has the dense head-major layout [L][B][heads][T][d] (or the
// forest is packed, which has no strides): what the kernels that address rows by item index need.
inline bool tv_layout_is_dense(const VerifyArgs& a) {
  if (a.tree.offsets != nullptr) return true;
  auto dense = [&](const Str3& s, int64_t heads, int64_t d) {
    return s.t == d && s.h == (int64_t)a.T * d && s.b == heads * a.T * d;
  };
  return dense(a.lay.qk, a.Hk, a.dk) && dense(a.lay.v, a.H, a.dv) && dense(a.lay.gate, a.H, 1) &&
         dense(a.lay.out, a.H, a.dv);
}

// Index of the q/k item (layer, request, key head) that state item (layer, request, head) reads.
__host__ __device__ inline int tv_qk_item(int item, int H, int Hk) {
  if (Hk == H) return item;
  const int lb = item / H, h = item - lb * H;
  return lb * Hk + h / (H / Hk);
}

// Where the rows of work item (layer l, request b, head h) live: element offsets of node 0 and
// the distance between consecutive nodes, per tensor class.  Dense or strided layout: from the
// resolved strides.  Packed forest: request b owns rows [offsets[b], offsets[b+1]) of every
// (layer, head) plane of `capacity` rows; its metadata slab is still T entries wide.
struct ItemRows {
  size_t qk0, v0, g0, o0;          // first element of node 0 in q/k | v | alpha/beta | O/U
  int64_t qk_rs, v_rs, g_rs, o_rs; // elements from one node to the next
  size_t meta0;                    // first entry in the metadata arrays
  int n;                           // real nodes of this item
};
__device__ inline ItemRows tv_item_rows(const TreeDev& t, const Layout& lay, int item, int B, int H, int Hk,
                                        int T, int dk, int dv) {
  ItemRows r;
  const int lb = item / H, h = item - lb * H;
  const int l = lb / B, b = lb - l * B;
  const int hk = Hk == H ? h : h / (H / Hk);
  if (t.offsets == nullptr) {
    r.qk0 = (size_t)((int64_t)lb * lay.qk.b + (int64_t)hk * lay.qk.h);
    r.v0 = (size_t)((int64_t)lb * lay.v.b + (int64_t)h * lay.v.h);
    r.g0 = (size_t)((int64_t)lb * lay.gate.b + (int64_t)h * lay.gate.h);
    r.o0 = (size_t)((int64_t)lb * lay.out.b + (int64_t)h * lay.out.h);
    r.qk_rs = lay.qk.t; r.v_rs = lay.v.t; r.g_rs = lay.gate.t; r.o_rs = lay.out.t;
    r.meta0 = (size_t)(t.n_trees == 1 ? 0 : b) * T;
    r.n = T;
  } else {
    const int off = t.offsets[b];
    r.n = t.offsets[b + 1] - off;
    const size_t node0 = (size_t)(l * H + h) * t.capacity + off;
    r.qk0 = ((size_t)(l * Hk + hk) * t.capacity + off) * dk;
    r.v0 = node0 * dv;
    r.g0 = node0;
    r.o0 = node0 * dv;
    r.qk_rs = dk; r.v_rs = dv; r.g_rs = 1; r.o_rs = dv;
    r.meta0 = (size_t)b * T;
  }
  return r;
}

void tv_set_cuda_error(cudaError_t e);

// Launchers (each returns a tv_status; all work is asynchronous on `stream`).
int tv_launch_verify_simt(const VerifyArgs& a, cudaStream_t stream);
int tv_launch_commit(const CommitArgs& a, const CommitLayers& layers, cudaStream_t stream);
int tv_launch_tree_meta(const int32_t* parent_mapped, int32_t n_trees, int32_t n, uint64_t* anc,
                        int32_t* depth, int32_t* parent_dev, int32_t* status, const int32_t* offsets_mapped,
                        int32_t* offsets_dev, int32_t depth_bound, int32_t generation, cudaStream_t stream);
// Host parents carried in the kernel parameters (small tree sets): no staging, no read over the bus.
bool tv_tree_meta_fits_params(int32_t n_trees, int32_t n, bool has_offsets);
int tv_launch_tree_meta_params(const int32_t* parent_host, int32_t n_trees, int32_t n, uint64_t* anc,
                               int32_t* depth, int32_t* parent_dev, int32_t* status, const int32_t* offsets_host,
                               int32_t* offsets_dev, cudaStream_t stream);
bool tv_verify_tc_supports(const VerifyArgs& a);
int tv_launch_verify_tc(const VerifyArgs& a, int32_t* status, cudaStream_t stream);
bool tv_verify_tc_delta_supports(const VerifyArgs& a);
int tv_launch_verify_tc_delta(const VerifyArgs& a, int32_t* status, cudaStream_t stream);
bool tv_verify_tc_delta128_supports(const VerifyArgs& a);   // 64 < T <= 128, dense layout
int tv_launch_verify_tc_delta128(const VerifyArgs& a, int32_t* status, cudaStream_t stream);

#define TV_CUDA_TRY(expr)                 \
  do {                                    \
    cudaError_t e__ = (expr);             \
    if (e__ != cudaSuccess) {             \
      tv_set_cuda_error(e__);             \
      return TV_ERR_CUDA;                 \
    }                                     \
  } while (0)
