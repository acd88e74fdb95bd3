// Device-side tree metadata (Section IV-A Table II: Anc(i), depth; Section IV-C "Round-level
// topology preprocessing"): one CTA per tree reads the parent array from pinned host memory
// and writes the strict-ancestor masks, depths and a device copy of the parents.  Nodes are
// indexed parent before child, so walking parent links from node i visits exactly Anc(i).
#include "tv_internal.h"
#include "tv_tc_common.cuh"

namespace {

__global__ void __launch_bounds__(TV_MAX_NODES)
tree_meta_kernel(const int32_t* __restrict__ parent, int32_t n, uint64_t* __restrict__ anc,
                 int32_t* __restrict__ depth, int32_t* __restrict__ parent_dev, int32_t* status,
                 const int32_t* __restrict__ offsets, int32_t* __restrict__ offsets_dev,
                 int32_t depth_bound, int32_t generation) {
  __shared__ int32_t par_s[TV_MAX_NODES];
  const int t = blockIdx.x, i = threadIdx.x;
  // This kernel is itself launched as a dependent of the kernels in front of it.  The parents and
  // offsets may be their output (a forest built on the device), and they may still be reading the
  // metadata of the previous upload: nothing is read or written before they have finished.
  tvtc::grid_dependency_wait();
  // A kernel launched behind this one may be scheduled now and set itself up; it waits for this
  // grid to finish before it reads the metadata.  Released only after the wait above, so that a
  // dependent never runs beside anything older than this grid (the library's kernels read data
  // that an older kernel may write -- the state -- before their own wait).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (i < n) {
    // host-built trees are validated there; device-built ones (tv_forest_upload_device) are not:
    // an out-of-range parent is treated as a child of the virtual root so the walk stays in bounds
    const int p = parent[(size_t)t * n + i];
    par_s[i] = (p < -1 || p >= i) ? -1 : p;
  }
  // packed forest: the row offsets travel with the parents (tree t copies entry t, the last
  // tree also the end marker)
  int32_t off0 = 0, off1 = 0;
  const bool copy_offsets = offsets != nullptr && i == 0, last_tree = t == (int)gridDim.x - 1;
  if (copy_offsets) {
    off0 = offsets[t];
    if (last_tree) off1 = offsets[t + 1];
  }
  __syncthreads();
  uint64_t w0 = 0, w1 = 0;
  int d = 0;
  // -1 <= parent[j] < j holds by now, so the walk ends within n steps.  The caller's depth bound
  // picked the kernels that will read these masks: a node deeper than that keeps its nearest
  // depth_bound ancestors only (every mask then fits those kernels' tables) and the upload is
  // marked as failed -- status[1] receives the generation of this upload (all CTAs write the same value),
  // which needs no clearing and so no ordering between the CTAs of this grid.
  int p = i < n ? par_s[i] : -1;
  for (; p >= 0 && d < depth_bound; p = par_s[p]) {
    if (p < 64) w0 |= 1ull << p; else w1 |= 1ull << (p - 64);
    ++d;
  }
  if (t == 0 && i == 0) *status = 0;
  if (copy_offsets) {
    offsets_dev[t] = off0;
    if (last_tree) offsets_dev[t + 1] = off1;
  }
  if (i >= n) return;
  if (p >= 0) atomicExch(status + 1, generation);
  const size_t o = (size_t)t * n + i;
  anc[2 * o] = w0;
  anc[2 * o + 1] = w1;
  depth[o] = d;
  parent_dev[o] = par_s[i];
}

// The same derivation with the parents carried in the kernel's PARAMETERS (one byte per node,
// -1..127), for tree sets small enough to fit: the launch itself brings the data, so the kernel
// does not start with a read over the bus.
template <int NB>
struct ParentBytes {
  int8_t p[NB];
};
struct OffsetWords {
  int32_t o[TV_MAX_NODES + 1 + 3];   // up to 128 requests + end marker
};

template <int NB>
__global__ void __launch_bounds__(TV_MAX_NODES)
tree_meta_param_kernel(const __grid_constant__ ParentBytes<NB> pb, const __grid_constant__ OffsetWords off,
                       int32_t has_offsets, int32_t n, uint64_t* __restrict__ anc, int32_t* __restrict__ depth,
                       int32_t* __restrict__ parent_dev, int32_t* status, int32_t* __restrict__ offsets_dev) {
  __shared__ int32_t par_s[TV_MAX_NODES];
  const int t = blockIdx.x, i = threadIdx.x;
  if (i < n) par_s[i] = pb.p[t * n + i];
  __syncthreads();
  uint64_t w0 = 0, w1 = 0;
  int d = 0;
  for (int p = i < n ? par_s[i] : -1; p >= 0 && d < n; p = par_s[p]) {
    if (p < 64) w0 |= 1ull << p; else w1 |= 1ull << (p - 64);
    ++d;
  }
  // Everything above read the kernel's parameters only.  The kernels in front on the stream may
  // still be reading the metadata of the previous upload (this kernel is launched as their
  // dependent): nothing is written before they have finished.
  tvtc::grid_dependency_wait();
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // after the wait, as in the kernel above
  if (t == 0 && i == 0) *status = 0;
  if (has_offsets && i == 0) {
    offsets_dev[t] = off.o[t];
    if (t == (int)gridDim.x - 1) offsets_dev[t + 1] = off.o[t + 1];
  }
  if (i >= n) return;
  const size_t o = (size_t)t * n + i;
  anc[2 * o] = w0;
  anc[2 * o + 1] = w1;
  depth[o] = d;
  parent_dev[o] = par_s[i];
}

template <int NB>
int launch_param(const int32_t* parent_host, int32_t n_trees, int32_t n, uint64_t* anc, int32_t* depth,
                 int32_t* parent_dev, int32_t* status, const int32_t* offsets_host, int32_t* offsets_dev,
                 cudaStream_t stream) {
  ParentBytes<NB> pb;
  const int nn = n_trees * n;
  for (int i = 0; i < nn; ++i) pb.p[i] = (int8_t)parent_host[i];   // validated: -1 <= parent < 128
  OffsetWords off;
  if (offsets_host)
    for (int i = 0; i <= n_trees; ++i) off.o[i] = offsets_host[i];
  TV_CUDA_TRY(tvtc::launch_dependent(tree_meta_param_kernel<NB>, n_trees, TV_MAX_NODES, 0, stream, pb, off,
                                     (int32_t)(offsets_host != nullptr), n, anc, depth, parent_dev, status,
                                     offsets_dev));
  return TV_OK;
}

}  // namespace

bool tv_tree_meta_fits_params(int32_t n_trees, int32_t n, bool has_offsets) {
  return (int64_t)n_trees * n <= 16384 && (!has_offsets || n_trees <= TV_MAX_NODES);
}

int tv_launch_tree_meta_params(const int32_t* parent_host, int32_t n_trees, int32_t n, uint64_t* anc,
                               int32_t* depth, int32_t* parent_dev, int32_t* status, const int32_t* offsets_host,
                               int32_t* offsets_dev, cudaStream_t stream) {
  const int nn = n_trees * n;
  if (nn <= 2048)
    return launch_param<2048>(parent_host, n_trees, n, anc, depth, parent_dev, status, offsets_host, offsets_dev,
                              stream);
  return launch_param<16384>(parent_host, n_trees, n, anc, depth, parent_dev, status, offsets_host, offsets_dev,
                             stream);
}

int tv_launch_tree_meta(const int32_t* parent_mapped, int32_t n_trees, int32_t n, uint64_t* anc,
                        int32_t* depth, int32_t* parent_dev, int32_t* status, const int32_t* offsets_mapped,
                        int32_t* offsets_dev, int32_t depth_bound, int32_t generation, cudaStream_t stream) {
  TV_CUDA_TRY(tvtc::launch_dependent(tree_meta_kernel, n_trees, TV_MAX_NODES, 0, stream, parent_mapped, n, anc, depth,
                                     parent_dev, status, offsets_mapped, offsets_dev, depth_bound, generation));
  return TV_OK;
}
