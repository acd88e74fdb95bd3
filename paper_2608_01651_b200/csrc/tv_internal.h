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

struct VerifyArgs {
  TreeDev tree;
  int32_t L, B, H, T, dk, dv, rule, bf16;
  int32_t Hk;  // q/k heads (H % Hk == 0); state head h reads q/k head h / (H / Hk)
  const float* S_pre;
  const void* q;
  const void* k;
  const void* v;
  const float* alpha;
  const float* beta;
  float* O;
  float* U;
};

struct CommitArgs {
  TreeDev tree;
  int32_t L, B, H, T, dk, dv, rule, bf16;
  int32_t Hk;
  const int32_t* accepted;
  const float* S_pre;
  const void* k;
  const void* v;
  const float* alpha;
  const float* beta;
  const float* U;
  float* S_new;
};

// Index of the q/k item (layer, request, key head) that state item (layer, request, head) reads.
__host__ __device__ inline int tv_qk_item(int item, int H, int Hk) {
  if (Hk == H) return item;
  const int lb = item / H, h = item - lb * H;
  return lb * Hk + h / (H / Hk);
}

// Where the rows of work item (layer l, request b, head h) live.  Dense layout: every item owns a
// slab of T rows.  Packed forest: request b owns rows [offsets[b], offsets[b+1]) of every
// (layer, head) plane of `capacity` rows; its metadata slab is still T entries wide.
struct ItemRows {
  size_t node0;   // first row in v / alpha / beta / O / U
  size_t qk0;     // first row in q / k
  size_t meta0;   // first entry in the metadata arrays
  int n;          // real nodes of this item
};
__device__ inline ItemRows tv_item_rows(const TreeDev& t, int item, int B, int H, int Hk, int T) {
  ItemRows r;
  const int lb = item / H, h = item - lb * H;
  const int l = lb / B, b = lb - l * B;
  const int hk = Hk == H ? h : h / (H / Hk);
  if (t.offsets == nullptr) {
    r.node0 = (size_t)item * T;
    r.qk0 = (size_t)(lb * Hk + hk) * T;
    r.meta0 = (size_t)(t.n_trees == 1 ? 0 : b) * T;
    r.n = T;
  } else {
    const int off = t.offsets[b];
    r.n = t.offsets[b + 1] - off;
    r.node0 = (size_t)(l * H + h) * t.capacity + off;
    r.qk0 = (size_t)(l * Hk + hk) * t.capacity + off;
    r.meta0 = (size_t)b * T;
  }
  return r;
}

void tv_set_cuda_error(cudaError_t e);

// Launchers (each returns a tv_status; all work is asynchronous on `stream`).
int tv_launch_verify_simt(const VerifyArgs& a, cudaStream_t stream);
int tv_launch_commit(const CommitArgs& a, cudaStream_t stream);
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
