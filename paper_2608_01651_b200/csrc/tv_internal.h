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
  int32_t* d_status = nullptr;  // device status word (0 = ok), cleared by every upload
  bool uploaded = false;
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

void tv_set_cuda_error(cudaError_t e);

// Launchers (each returns a tv_status; all work is asynchronous on `stream`).
int tv_launch_verify_simt(const VerifyArgs& a, cudaStream_t stream);
int tv_launch_commit(const CommitArgs& a, cudaStream_t stream);
int tv_launch_tree_meta(const int32_t* parent_mapped, int32_t n_trees, int32_t n, uint64_t* anc,
                        int32_t* depth, int32_t* parent_dev, int32_t* status, cudaStream_t stream);
bool tv_verify_tc_supports(const VerifyArgs& a);
int tv_launch_verify_tc(const VerifyArgs& a, int32_t* status, cudaStream_t stream);
bool tv_verify_tc_delta_supports(const VerifyArgs& a);
int tv_launch_verify_tc_delta(const VerifyArgs& a, int32_t* status, cudaStream_t stream);

#define TV_CUDA_TRY(expr)                 \
  do {                                    \
    cudaError_t e__ = (expr);             \
    if (e__ != cudaSuccess) {             \
      tv_set_cuda_error(e__);             \
      return TV_ERR_CUDA;                 \
    }                                     \
  } while (0)
