// tv_tree_verify_static: tree verification for callers that must not allocate.
//
// Who cannot allocate: code that runs where cudaMalloc is forbidden or unsafe -- inside a
// CUDA-graph capture region or a memory-pool-managed serving loop whose device memory was
// fully carved up at start-up, plug-ins loaded into a process that owns the allocator, and
// latency-critical paths where an allocation (an implicit device synchronisation) is not
// acceptable.  The regular path allocates in tv_tree_build / tv_tree_upload (host vectors,
// the device mirror of the tree metadata, pinned staging).  Here the metadata lives in a
// file-scope device array instead, the parent arrays are read from DEVICE memory (as a
// drafter running on the GPU leaves them), and nothing is allocated or freed.
#include "tv_internal.h"

namespace {

constexpr int kMaxTrees = TV_STATIC_MAX_TREES;
constexpr size_t kNodes = (size_t)kMaxTrees * TV_MAX_NODES;
constexpr size_t kAncBytes = kNodes * 2 * sizeof(uint64_t);
constexpr size_t kI32Bytes = kNodes * sizeof(int32_t);
constexpr size_t kScratchBytes = kAncBytes + 2 * kI32Bytes + 256;   // masks | depths | parents | status

// The scratch.  Every GPU that loads the library holds these 384 KiB until the process exits.
// In host code this name is only a stand-in for the symbol: the device address comes from
// cudaGetSymbolAddress below and is what the kernels receive.
static __device__ __align__(256) unsigned char g_static_tree[kScratchBytes];

// Same derivation as the regular metadata kernel, but the parents come from device memory and
// cannot have been checked by the host: a parent outside [-1, i) is reported in the status
// word and treated as "child of the virtual root", so the kernels that follow stay in bounds.
__global__ void __launch_bounds__(TV_MAX_NODES)
tree_meta_static_kernel(const int32_t* __restrict__ parent, int32_t n, uint64_t* __restrict__ anc,
                        int32_t* __restrict__ depth, int32_t* __restrict__ parent_dev,
                        int32_t* scratch_status, int32_t* user_status) {
  __shared__ int32_t par_s[TV_MAX_NODES];
  const int t = blockIdx.x, i = threadIdx.x;
  // a verify kernel launched behind this one may be scheduled now and set itself up; it waits
  // for this grid to finish before it reads global memory
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  bool bad = false;
  if (i < n) {
    int p = parent[(size_t)t * n + i];
    if (p < -1 || p >= i) {
      bad = true;
      p = -1;
    }
    par_s[i] = p;
  }
  // the status word of the launch that is about to read this metadata starts at zero
  if (t == 0 && i == 0) *scratch_status = 0;
  if (__syncthreads_or(bad) && i == 0 && user_status) atomicExch(user_status, (int)TV_ERR_INVALID_TREE);
  if (i >= n) return;
  uint64_t w0 = 0, w1 = 0;
  int d = 0;
  for (int p = par_s[i]; p >= 0 && d < n; p = par_s[p]) {
    if (p < 64) w0 |= 1ull << p; else w1 |= 1ull << (p - 64);
    ++d;
  }
  const size_t o = (size_t)t * n + i;
  anc[2 * o] = w0;
  anc[2 * o + 1] = w1;
  depth[o] = d;
  parent_dev[o] = par_s[i];
}

// Forwards a device-side timeout of the verify kernel to the caller's status word.
__global__ void forward_status_kernel(const int32_t* scratch_status, int32_t* user_status) {
  const int s = *scratch_status;
  if (s != 0) atomicExch(user_status, s);
}

// Device address of the scratch, looked up once per device with that device current.
unsigned char* scratch_address(int dev, cudaError_t* err) {
  constexpr int kMaxDevices = 64;
  static unsigned char* table[kMaxDevices] = {};
  *err = cudaSuccess;
  if (dev < 0 || dev >= kMaxDevices) {
    *err = cudaErrorInvalidDevice;
    return nullptr;
  }
  if (!table[dev]) {
    unsigned char* ptr = nullptr;
    *err = cudaGetSymbolAddress((void**)&ptr, g_static_tree);
    if (*err != cudaSuccess) return nullptr;
    table[dev] = ptr;
  }
  return table[dev];
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

}  // namespace

extern "C" __attribute__((visibility("default")))
int tv_tree_verify_static(const int32_t* parent, int32_t n_trees, const tv_dims* d, const float* S_pre,
                          const void* q, const void* k, const void* v, const float* alpha,
                          const float* beta, float* O, float* U, int32_t* status, void* stream) {
  if (!parent || !d || !S_pre || !q || !k || !v || !alpha || !O) return TV_ERR_BAD_ARG;
  if (d->L < 1 || d->B < 1 || d->H < 1 || d->T < 1 || d->dk < 1 || d->dv < 1) return TV_ERR_BAD_ARG;
  if (d->rule != TV_GATED && d->rule != TV_GATED_DELTA) return TV_ERR_BAD_ARG;
  if (d->qkv_dtype != TV_F32 && d->qkv_dtype != TV_BF16) return TV_ERR_BAD_ARG;
  if (d->impl != TV_IMPL_AUTO && d->impl != TV_IMPL_SIMT && d->impl != TV_IMPL_TC) return TV_ERR_BAD_ARG;
  if (d->rule == TV_GATED_DELTA && !beta) return TV_ERR_BAD_ARG;
  if (n_trees != 1 && n_trees != d->B) return TV_ERR_BAD_ARG;
  if (d->Hk < 0 || d->Hk > d->H || (d->Hk > 0 && d->H % d->Hk != 0)) return TV_ERR_BAD_ARG;
  // beyond the fixed scratch: refuse, never spill into an allocation
  if (n_trees > kMaxTrees) return TV_ERR_TOO_LARGE;
  if (d->T > TV_MAX_NODES || d->dk > TV_MAX_DIM || d->dv > TV_MAX_DIM) return TV_ERR_UNSUPPORTED;
  if ((d->dk & 3) || (d->dv & 3)) return TV_ERR_UNSUPPORTED;
  if (d->qkv_dtype == TV_BF16 && ((d->dk & 7) || (d->dv & 7))) return TV_ERR_UNSUPPORTED;
  if ((int64_t)d->L * d->B * d->H > 0x7fffffffLL) return TV_ERR_UNSUPPORTED;
  if (!aligned16(S_pre) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(O) ||
      !aligned16(U) || ((uintptr_t)alpha & 3) || ((uintptr_t)beta & 3) || ((uintptr_t)parent & 3) ||
      ((uintptr_t)status & 3))
    return TV_ERR_BAD_ARG;

  int dev = 0;
  TV_CUDA_TRY(cudaGetDevice(&dev));
  cudaError_t err;
  unsigned char* base = scratch_address(dev, &err);
  if (!base) {
    tv_set_cuda_error(err);
    return TV_ERR_CUDA;
  }
  uint64_t* anc = reinterpret_cast<uint64_t*>(base);
  int32_t* depth = reinterpret_cast<int32_t*>(base + kAncBytes);
  int32_t* par_dev = reinterpret_cast<int32_t*>(base + kAncBytes + kI32Bytes);
  int32_t* scratch_status = reinterpret_cast<int32_t*>(base + kAncBytes + 2 * kI32Bytes);

  VerifyArgs a;
  a.tree.anc = anc;
  a.tree.depth = depth;
  a.tree.parent = par_dev;
  a.tree.n_trees = n_trees;
  a.tree.max_depth_all = TV_MAX_NODES - 1;   // not known on the host
  a.tree.offsets = nullptr;
  a.tree.capacity = 0;
  a.L = d->L; a.B = d->B; a.H = d->H; a.T = d->T; a.dk = d->dk; a.dv = d->dv;
  a.rule = d->rule; a.bf16 = d->qkv_dtype == TV_BF16; a.Hk = d->Hk ? d->Hk : d->H;
  a.S_pre = S_pre; a.q = q; a.k = k; a.v = v; a.alpha = alpha; a.beta = beta; a.O = O; a.U = U;
  const int lst = tv_resolve_layout(d, false, &a.lay);
  if (lst != TV_OK) return lst;
  // every refusal comes before the first launch: an error return has touched nothing, not even
  // the scratch that all calls share
  const bool tc_gated = tv_verify_tc_supports(a);
  if (d->impl == TV_IMPL_TC && !tc_gated) return TV_ERR_UNSUPPORTED;

  cudaStream_t s = (cudaStream_t)stream;
  tree_meta_static_kernel<<<n_trees, TV_MAX_NODES, 0, s>>>(parent, d->T, anc, depth, par_dev,
                                                          scratch_status, status);
  TV_CUDA_TRY(cudaGetLastError());
  int st;
  if (tc_gated && d->impl != TV_IMPL_SIMT) st = tv_launch_verify_tc(a, scratch_status, s);
  else st = tv_launch_verify_simt(a, s);
  if (st != TV_OK) return st;
  if (status) {
    forward_status_kernel<<<1, 1, 0, s>>>(scratch_status, status);
    TV_CUDA_TRY(cudaGetLastError());
  }
  return TV_OK;
}
