// Tree verification, general fp32 SIMT kernel (any T <= 128, dk, dv <= 128,
// f32 or bf16 operands, gated and delta rules).  All arithmetic is fp32 FMA,
// so this kernel also serves the all-fp32 workloads with a 1e-5 bound; the
// tensor-core kernel takes the bf16 dk = dv = 128 shapes.
//
// One CTA per (layer, request, head), following Theorem 1 (Eq. 2) in the
// factorised form of Eq. 4 / Lemma 2 (Eq. 5):
//   1. P_i from the ancestor mask (Table II).
//   2. S_pre staged once in shared memory, transposed to [dk][dv].
//   3. dense part on a register-tiled GEMM:  B0 = D_P (Q S_pre^T)  -> O,
//      delta rule also  R = D_beta (V - D_P K S_pre^T)             -> smem U.
//   4. delta rule: (I + G) U = R solved level by level (nodes of equal depth
//      are independent; G_ij != 0 only for strict ancestors j, Lemma 2), which
//      is the finite polynomial of Lemma 3 evaluated by substitution.
//   5. sparse part: O_i += sum_{j in Anc(i)+{i}} (P_i/P_j)(q_i.k_j) u_j, one
//      warp per node walking the set bits of its mask from the node upwards;
//      the decay ratio is the running product of alpha, never a division.
// No per-node state is formed and nothing but O (and U on request) is written.
#include <cuda_bf16.h>

#include "tv_internal.h"
#include "tv_tc_common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kSLD = TV_MAX_DIM + 4;  // row stride of the transposed state
constexpr int kALD = 33;              // row stride of the staged operand chunk
constexpr int kKC = 32;               // k-chunk of the dense pass

template <bool BF16>
__device__ __forceinline__ float load_elem(const void* base, size_t idx) {
  if (BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(base)[idx]);
  return reinterpret_cast<const float*>(base)[idx];
}

// 4 consecutive elements starting at idx (idx % 4 == 0) widened to float.
template <bool BF16>
__device__ __forceinline__ float4 load4(const void* base, size_t idx) {
  if (BF16) {
    const uint2 r = *reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(base) + idx);
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&r.x);
    const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&r.y);
    const float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
    return make_float4(fa.x, fa.y, fb.x, fb.y);
  }
  return *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(base) + idx);
}

// Removes and returns the highest set bit of the 128-bit set (m1:m0); -1 if empty.
__device__ __forceinline__ int pop_highest(uint64_t& m0, uint64_t& m1) {
  if (m1) {
    const int b = 63 - __clzll((long long)m1);
    m1 &= ~(1ull << b);
    return 64 + b;
  }
  if (m0) {
    const int b = 63 - __clzll((long long)m0);
    m0 &= ~(1ull << b);
    return b;
  }
  return -1;
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

struct Smem {
  float* S_T;       // [dk][kSLD]
  float* U_s;       // [T][dv]      (delta rule)
  float* A_s;       // [128][kALD]
  uint64_t* anc_s;  // [T][2]
  float* P_s;       // [T]
  float* alpha_s;   // [T]
  float* beta_s;    // [T]
  int* depth_s;     // [T]
};

// Dense pass: acc[i][v] = sum_k A[i][k] S_pre[v][k], then an epilogue per mode.
//   mode 0 (A = Q): O[i][v] = P_i acc
//   mode 1 (A = K): U_s[i][v] = beta_i (v_i[v] - P_i acc)
template <bool BF16, int MODE>
__device__ __forceinline__ void dense_pass(const VerifyArgs& a, const Smem& sm, const void* A,
                                           const ItemRows& rows, int T, float* Og) {
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int dk = a.dk, dv = a.dv;
  float acc[8][8];
#pragma unroll
  for (int m = 0; m < 8; ++m)
#pragma unroll
    for (int n = 0; n < 8; ++n) acc[m][n] = 0.f;

  for (int k0 = 0; k0 < dk; k0 += kKC) {
    __syncthreads();
    for (int idx = tid; idx < TV_MAX_NODES * kKC; idx += kThreads) {
      const int i = idx >> 5, kk = idx & 31;
      float x = 0.f;
      if (i < T && k0 + kk < dk) x = load_elem<BF16>(A, rows.qk0 + (size_t)i * rows.qk_rs + k0 + kk);
      sm.A_s[i * kALD + kk] = x;
    }
    __syncthreads();
    const int kmax = ty * 8 < T ? min(kKC, dk - k0) : 0;  // skip row tiles past the tree
    for (int kk = 0; kk < kmax; ++kk) {
      float av[8];
#pragma unroll
      for (int m = 0; m < 8; ++m) av[m] = sm.A_s[(ty * 8 + m) * kALD + kk];
      const float* srow = sm.S_T + (size_t)(k0 + kk) * kSLD;
      const float4 s0 = *reinterpret_cast<const float4*>(srow + tx * 4);
      const float4 s1 = *reinterpret_cast<const float4*>(srow + 64 + tx * 4);
      const float sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
      for (int m = 0; m < 8; ++m)
#pragma unroll
        for (int n = 0; n < 8; ++n) acc[m][n] = fmaf(av[m], sv[n], acc[m][n]);
    }
  }
#pragma unroll
  for (int m = 0; m < 8; ++m) {
    const int i = ty * 8 + m;
    if (i >= T) continue;
    const float Pi = sm.P_s[i];
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int v0 = half * 64 + tx * 4;
      if (v0 >= dv) continue;
      float4 r = make_float4(Pi * acc[m][half * 4 + 0], Pi * acc[m][half * 4 + 1],
                             Pi * acc[m][half * 4 + 2], Pi * acc[m][half * 4 + 3]);
      if (MODE == 0) {
        *reinterpret_cast<float4*>(Og + (size_t)i * rows.o_rs + v0) = r;
      } else {
        const float4 vv = load4<BF16>(a.v, rows.v0 + (size_t)i * rows.v_rs + v0);
        const float be = sm.beta_s[i];
        r = make_float4(be * (vv.x - r.x), be * (vv.y - r.y), be * (vv.z - r.z), be * (vv.w - r.w));
        *reinterpret_cast<float4*>(sm.U_s + (size_t)i * dv + v0) = r;
      }
    }
  }
}

template <bool BF16, bool DELTA>
__global__ void __launch_bounds__(kThreads) verify_simt_kernel(VerifyArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // Dependent launch on both sides: this kernel reads nothing -- the tree metadata may come from
  // the kernel in front -- before that kernel is done; the kernel behind it may set itself up from
  // then on (the library's kernels read nothing this one writes before their own wait, and a
  // dependent released after the wait never runs beside anything older than this grid).
  tvtc::grid_dependency_wait();
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int dk = a.dk, dv = a.dv;
  const int item = blockIdx.x;
  const ItemRows rows = tv_item_rows(a.tree, a.lay, item, a.B, a.H, a.Hk, a.T, a.dk, a.dv);
  const int T = rows.n;   // real nodes of this item (the whole slab unless the forest is packed)
  Smem sm;
  {
    unsigned char* p = smem_raw;
    sm.S_T = reinterpret_cast<float*>(p);  p += sizeof(float) * TV_MAX_DIM * kSLD;
    sm.A_s = reinterpret_cast<float*>(p);  p += sizeof(float) * TV_MAX_NODES * kALD + 16;
    p = reinterpret_cast<unsigned char*>(((uintptr_t)p + 15) & ~(uintptr_t)15);
    sm.anc_s = reinterpret_cast<uint64_t*>(p);  p += sizeof(uint64_t) * 2 * TV_MAX_NODES;
    sm.P_s = reinterpret_cast<float*>(p);  p += sizeof(float) * TV_MAX_NODES;
    sm.alpha_s = reinterpret_cast<float*>(p);  p += sizeof(float) * TV_MAX_NODES;
    sm.beta_s = reinterpret_cast<float*>(p);  p += sizeof(float) * TV_MAX_NODES;
    sm.depth_s = reinterpret_cast<int*>(p);  p += sizeof(int) * TV_MAX_NODES;
    sm.U_s = reinterpret_cast<float*>(p);  // only with DELTA
  }
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* Sg = a.S_pre + (size_t)item * dv * dk;
  float* Og = a.O + rows.o0;

  // 1. metadata and path decay P_i
  if (tid < T) {
    const uint64_t* m = a.tree.anc + (rows.meta0 + tid) * 2;
    sm.anc_s[2 * tid] = m[0];
    sm.anc_s[2 * tid + 1] = m[1];
    sm.alpha_s[tid] = a.alpha[rows.g0 + (size_t)tid * rows.g_rs];
    sm.beta_s[tid] = DELTA ? a.beta[rows.g0 + (size_t)tid * rows.g_rs] : 0.f;
    sm.depth_s[tid] = a.tree.depth[rows.meta0 + tid];
  }
  __syncthreads();
  if (tid < T) {
    uint64_t m0 = sm.anc_s[2 * tid], m1 = sm.anc_s[2 * tid + 1];
    float P = sm.alpha_s[tid];
    for (int j = pop_highest(m0, m1); j >= 0; j = pop_highest(m0, m1)) P *= sm.alpha_s[j];
    sm.P_s[tid] = P;
  }
  // 2. stage S_pre transposed: S_T[k][v]
  {
    const int dk4 = dk >> 2, n4 = dv * dk4;
    for (int i = tid; i < n4; i += kThreads) {
      const int v = i / dk4, c4 = i - v * dk4;
      const float4 t = reinterpret_cast<const float4*>(Sg)[i];
      float* d = sm.S_T + (size_t)(c4 * 4) * kSLD + v;
      d[0] = t.x; d[kSLD] = t.y; d[2 * kSLD] = t.z; d[3 * kSLD] = t.w;
    }
  }
  __syncthreads();

  // 3. dense part
  dense_pass<BF16, 0>(a, sm, a.q, rows, T, Og);
  if (DELTA) dense_pass<BF16, 1>(a, sm, a.k, rows, T, Og);
  __syncthreads();

  const int nk = dk >> 2;  // lanes holding 4 consecutive k elements
  // 4. delta rule: level-ordered substitution for (I + G) U = R
  if (DELTA) {
    int dmax = 0;
    for (int i = 0; i < T; ++i) dmax = max(dmax, sm.depth_s[i]);
    for (int lev = 1; lev <= dmax; ++lev) {
      for (int i = warp; i < T; i += kWarps) {
        if (sm.depth_s[i] != lev) continue;
        float4 ki = make_float4(0.f, 0.f, 0.f, 0.f);
        if (lane < nk) ki = load4<BF16>(a.k, rows.qk0 + (size_t)i * rows.qk_rs + lane * 4);
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        uint64_t m0 = sm.anc_s[2 * i], m1 = sm.anc_s[2 * i + 1];
        float w = sm.alpha_s[i];  // P_i / P_parent(i)
        for (int j = pop_highest(m0, m1); j >= 0; j = pop_highest(m0, m1)) {
          float4 kj = make_float4(0.f, 0.f, 0.f, 0.f);
          if (lane < nk) kj = load4<BF16>(a.k, rows.qk0 + (size_t)j * rows.qk_rs + lane * 4);
          const float dot = warp_sum(ki.x * kj.x + ki.y * kj.y + ki.z * kj.z + ki.w * kj.w);
          const float g = w * dot;
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            const int c = lane + 32 * x;
            if (c < dv) acc[x] = fmaf(g, sm.U_s[(size_t)j * dv + c], acc[x]);
          }
          w *= sm.alpha_s[j];
        }
        const float be = sm.beta_s[i];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const int c = lane + 32 * x;
          if (c < dv) sm.U_s[(size_t)i * dv + c] -= be * acc[x];
        }
      }
      __syncthreads();
    }
  }

  // 5. sparse readout: O_i += sum_j C_ij u_j
  for (int i = warp; i < T; i += kWarps) {
    float4 qi = make_float4(0.f, 0.f, 0.f, 0.f);
    if (lane < nk) qi = load4<BF16>(a.q, rows.qk0 + (size_t)i * rows.qk_rs + lane * 4);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    uint64_t m0 = sm.anc_s[2 * i], m1 = sm.anc_s[2 * i + 1];
    float w = 1.f;
    int j = i;
    while (j >= 0) {
      float4 kj = make_float4(0.f, 0.f, 0.f, 0.f);
      if (lane < nk) kj = load4<BF16>(a.k, rows.qk0 + (size_t)j * rows.qk_rs + lane * 4);
      const float dot = warp_sum(qi.x * kj.x + qi.y * kj.y + qi.z * kj.z + qi.w * kj.w);
      const float c = w * dot;
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const int ch = lane + 32 * x;
        if (ch < dv) {
          const float u = DELTA ? sm.U_s[(size_t)j * dv + ch] : load_elem<BF16>(a.v, rows.v0 + (size_t)j * rows.v_rs + ch);
          acc[x] = fmaf(c, u, acc[x]);
        }
      }
      w *= sm.alpha_s[j];
      j = pop_highest(m0, m1);
    }
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const int ch = lane + 32 * x;
      if (ch < dv) Og[(size_t)i * rows.o_rs + ch] += acc[x];
    }
  }

  // 6. corrections on request
  if (a.U) {
    float* Ug = a.U + rows.o0;
    for (int i = tid; i < T * dv; i += kThreads) {
      const int t = i / dv, c = i - t * dv;
      Ug[(size_t)t * rows.o_rs + c] = DELTA ? sm.U_s[i] : load_elem<BF16>(a.v, rows.v0 + (size_t)t * rows.v_rs + c);
    }
  }
}

size_t smem_bytes(bool delta) {
  size_t b = sizeof(float) * TV_MAX_DIM * kSLD + sizeof(float) * TV_MAX_NODES * kALD + 32 +
             sizeof(uint64_t) * 2 * TV_MAX_NODES + 4 * sizeof(float) * TV_MAX_NODES;
  if (delta) b += sizeof(float) * TV_MAX_NODES * TV_MAX_DIM;
  return b;
}

template <bool BF16, bool DELTA>
int launch(const VerifyArgs& a, cudaStream_t stream) {
  const size_t smem = smem_bytes(DELTA);
  auto kern = verify_simt_kernel<BF16, DELTA>;
  static thread_local int configured_dev[4] = {-1, -1, -1, -1};
  int dev = 0;
  TV_CUDA_TRY(cudaGetDevice(&dev));
  int& slot = configured_dev[(BF16 ? 1 : 0) + (DELTA ? 2 : 0)];
  if (slot != dev) {
    TV_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    slot = dev;
  }
  TV_CUDA_TRY(tvtc::launch_dependent(kern, a.L * a.B * a.H, kThreads, smem, stream, a));
  return TV_OK;
}

}  // namespace

int tv_launch_verify_simt(const VerifyArgs& a, cudaStream_t stream) {
  const bool delta = a.rule == TV_GATED_DELTA;
  if (a.bf16) return delta ? launch<true, true>(a, stream) : launch<true, false>(a, stream);
  return delta ? launch<false, true>(a, stream) : launch<false, false>(a, stream);
}
