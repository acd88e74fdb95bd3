// Batch-wide utility allocation (Section V-A): score every candidate node by the drafter's
// probability of its whole path, keep the root of every tree plus the highest-scoring nodes of the
// whole batch up to a fixed budget, count per request, and pack the kept nodes into the padded
// parent slabs and offsets of a packed forest (Section V-B) -- all on the device, with fixed
// shapes, so the selection can sit inside a GPU-resident round.
//
// Three small launches:
//   budget_rho_kernel     one CTA per request: rho_i = rho_parent * p_i in float32, level by level
//                         (parent before child, one rounding per edge), and a 32-bit sort key
//   budget_select_kernel  one CTA: 4-pass radix select of the budget-th largest key, ties taken in
//                         (request, node) order, then per-request counts and their prefix sums
//   budget_pack_kernel    one CTA per request: order-preserving compaction and parent renumbering
// The sizes are tiny (at most a few 10^4 candidates); the point is determinism and staying on the
// stream, not bandwidth.
#include "tv_internal.h"

namespace {

constexpr int kSelThreads = 1024;

__global__ void __launch_bounds__(TV_MAX_NODES)
budget_rho_kernel(const int32_t* __restrict__ parent, const float* __restrict__ p, int32_t Tc,
                  float* __restrict__ rho, uint32_t* __restrict__ key, int32_t* status) {
  __shared__ int32_t par_s[TV_MAX_NODES];
  __shared__ float rho_s[TV_MAX_NODES];
  __shared__ int maxd_s;
  const int b = blockIdx.x, i = threadIdx.x;
  if (i == 0) maxd_s = 0;
  int par = -1;
  float pi = 0.f;
  if (i < Tc) {
    par = parent[(size_t)b * Tc + i];
    pi = p[(size_t)b * Tc + i];
    if (par < -1 || par >= i || (i == 0 && par != -1)) {   // cannot be checked on the host
      par = -1;
      if (status) atomicExch(status, (int)TV_ERR_INVALID_TREE);
    }
    par_s[i] = par;
  }
  __syncthreads();
  int depth = 0;
  if (i < Tc) {
    for (int j = par; j >= 0 && depth < Tc; j = par_s[j]) ++depth;
    atomicMax(&maxd_s, depth);
  }
  __syncthreads();
  const int maxd = maxd_s;
  for (int d = 0; d <= maxd; ++d) {
    if (i < Tc && depth == d) rho_s[i] = par < 0 ? pi : __fmul_rn(rho_s[par], pi);
    __syncthreads();
  }
  if (i < Tc) {
    const float r = rho_s[i];
    rho[(size_t)b * Tc + i] = r;
    // non-negative floats order like their bit patterns; roots rank above everything
    key[(size_t)b * Tc + i] = i == 0 ? 0xffffffffu : (r >= 0.f ? __float_as_uint(r) : 0u);
  }
}

// Exclusive prefix sum of one int per thread over the CTA (kSelThreads threads).
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_tot, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int up = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += up;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = warp_tot[lane];
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += up;
    }
    warp_tot[lane] = wi - w;   // exclusive over warps
    if (lane == 31) *total = wi;
  }
  __syncthreads();
  return warp_tot[warp] + incl - v;
}

__global__ void __launch_bounds__(kSelThreads)
budget_select_kernel(const uint32_t* __restrict__ key, int32_t N, int32_t K, int32_t B, int32_t Tc,
                     uint8_t* __restrict__ keep, int32_t* __restrict__ counts, int32_t* __restrict__ offsets) {
  __shared__ int hist[256];
  __shared__ uint32_t prefix_s;
  __shared__ int need_s;
  __shared__ int warp_tot[32];
  __shared__ int total_s;
  __shared__ int cnt_s[kSelThreads];   // kept nodes per request (B <= kSelThreads)
  const int tid = threadIdx.x;
  cnt_s[tid] = 0;
  if (tid == 0) {
    prefix_s = 0;
    need_s = K;
  }
  // ---- the K-th largest key, one byte at a time from the top ----
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    const uint32_t prefix = prefix_s;
    for (int i = tid; i < N; i += kSelThreads) {
      const uint32_t k = key[i];
      if (pass == 0 || (k >> (shift + 8)) == prefix) atomicAdd(&hist[(k >> shift) & 255u], 1);
    }
    __syncthreads();
    // the digit whose bucket holds the need-th largest key: thread t looks at digit 255 - t and
    // at the number of keys in the higher buckets (a prefix sum over the CTA, not a serial walk)
    {
      const int need = need_s;
      const int mine = tid < 256 ? hist[255 - tid] : 0;
      const int above = block_exclusive_scan(mine, warp_tot, &total_s);
      if (tid < 256 && above < need && above + mine >= need) {
        prefix_s = (prefix << 8) | (uint32_t)(255 - tid);
        need_s = need - above;   // how many keys with this prefix still have to be taken
      }
    }
    __syncthreads();
  }
  const uint32_t tau = prefix_s;   // the threshold key
  const int need = need_s;         // number of keys == tau to take, in index order
  // ---- flags: everything above the threshold, and the first `need` keys equal to it ----
  const int chunk = (N + kSelThreads - 1) / kSelThreads;
  const int i0 = tid * chunk, i1 = min(N, i0 + chunk);
  int ties = 0;
  for (int i = i0; i < i1; ++i) ties += key[i] == tau;
  int before = block_exclusive_scan(ties, warp_tot, &total_s);
  for (int i = i0; i < i1; ++i) {
    const uint32_t k = key[i];
    bool take = k > tau;
    if (k == tau) take = before++ < need;
    keep[i] = take ? 1 : 0;
    if (take) atomicAdd(&cnt_s[i / Tc], 1);
  }
  __syncthreads();
  // ---- per-request counts and their exclusive prefix sums (B <= kSelThreads) ----
  const int c = tid < B ? cnt_s[tid] : 0;
  const int off = block_exclusive_scan(c, warp_tot, &total_s);
  if (tid < B) {
    counts[tid] = c;
    offsets[tid] = off;
  }
  if (tid == 0) offsets[B] = total_s;
}

__global__ void __launch_bounds__(TV_MAX_NODES)
budget_pack_kernel(const int32_t* __restrict__ parent, const uint8_t* __restrict__ keep,
                   const int32_t* __restrict__ offsets, int32_t B, int32_t Tc, int32_t budget,
                   int32_t* __restrict__ parent_packed, int32_t* __restrict__ node_id) {
  __shared__ int rank_s[TV_MAX_NODES];
  __shared__ int warp_tot[4];
  const int b = blockIdx.x, i = threadIdx.x, lane = i & 31, warp = i >> 5;
  const bool flag = i < Tc && keep[(size_t)b * Tc + i] != 0;
  const unsigned ballot = __ballot_sync(0xffffffffu, flag);
  if (lane == 0) warp_tot[warp] = __popc(ballot);
  __syncthreads();
  int rank = __popc(ballot & ((1u << lane) - 1u));
  for (int w = 0; w < warp; ++w) rank += warp_tot[w];
  const int count = warp_tot[0] + warp_tot[1] + warp_tot[2] + warp_tot[3];
  rank_s[i] = flag ? rank : -1;
  __syncthreads();
  if (flag) {
    int par = parent[(size_t)b * Tc + i];
    if (par < -1 || par >= i) par = -1;
    parent_packed[(size_t)b * Tc + rank] = par < 0 ? -1 : rank_s[par];   // -1 also if the parent was dropped
    node_id[offsets[b] + rank] = b * Tc + i;
  }
  if (i >= count && i < Tc) parent_packed[(size_t)b * Tc + i] = -1;       // padding of the slab
  if (b == 0)
    for (int j = offsets[B] + i; j < budget; j += TV_MAX_NODES) node_id[j] = -1;   // rows past the forest
}

}  // namespace

#define TV_API __attribute__((visibility("default")))

extern "C" {

TV_API size_t tv_budget_workspace_bytes(int32_t n_req, int32_t n_cand) {
  if (n_req < 1 || n_cand < 1) return 0;
  const size_t N = (size_t)n_req * n_cand;
  return ((N * sizeof(uint32_t) + 255) & ~(size_t)255) + ((N + 255) & ~(size_t)255);
}

TV_API int tv_budget_select(const int32_t* parent, const float* p_draft, int32_t n_req, int32_t n_cand,
                            int32_t budget, float* rho, int32_t* counts, int32_t* offsets,
                            int32_t* parent_packed, int32_t* node_id, void* workspace, int32_t* status,
                            void* stream) {
  if (!parent || !p_draft || !rho || !counts || !offsets || !parent_packed || !node_id || !workspace)
    return TV_ERR_BAD_ARG;
  if (n_req < 1 || n_cand < 1 || budget < n_req) return TV_ERR_BAD_ARG;
  if (n_cand > TV_MAX_NODES || n_req > kSelThreads) return TV_ERR_UNSUPPORTED;
  if (((uintptr_t)parent | (uintptr_t)p_draft | (uintptr_t)rho | (uintptr_t)counts | (uintptr_t)offsets |
       (uintptr_t)parent_packed | (uintptr_t)node_id | (uintptr_t)status) & 3)
    return TV_ERR_BAD_ARG;
  if ((uintptr_t)workspace & 15) return TV_ERR_BAD_ARG;
  const int32_t N = n_req * n_cand;
  const int32_t K = budget < N ? budget : N;
  uint32_t* key = reinterpret_cast<uint32_t*>(workspace);
  uint8_t* keep = reinterpret_cast<uint8_t*>(workspace) + (((size_t)N * sizeof(uint32_t) + 255) & ~(size_t)255);
  cudaStream_t s = (cudaStream_t)stream;
  budget_rho_kernel<<<n_req, TV_MAX_NODES, 0, s>>>(parent, p_draft, n_cand, rho, key, status);
  TV_CUDA_TRY(cudaGetLastError());
  budget_select_kernel<<<1, kSelThreads, 0, s>>>(key, N, K, n_req, n_cand, keep, counts, offsets);
  TV_CUDA_TRY(cudaGetLastError());
  budget_pack_kernel<<<n_req, TV_MAX_NODES, 0, s>>>(parent, keep, offsets, n_req, n_cand, budget, parent_packed,
                                                   node_id);
  TV_CUDA_TRY(cudaGetLastError());
  return TV_OK;
}

}  // extern "C"
