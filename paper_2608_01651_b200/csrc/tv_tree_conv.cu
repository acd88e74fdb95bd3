// Stage 1 of the per-layer pipeline (Section IV-C): tree-parallel causal depthwise convolution
// + bias + SiLU, optional q/k normalisation, gate preparation, and the head-major layout the
// verification kernels read -- one pass over the projected activations.
//
// The work is a gather along parent links with W taps per output and no reuse beyond the tile,
// so it is bound by HBM: x is read once, q/k/v are written once.  One CTA owns one
// (request, head, q|k|v) slice: T rows of d channels.  It stages the slice (plus the W-1 context
// rows) in shared memory with 16-byte streaming loads, derives each node's W tap rows from the
// parent array once, and then one warp per node row gathers the taps from shared memory, so a
// row's sum of squares (for the normalisation) is a warp reduction and the row leaves as one
// contiguous store.
#include <cuda_bf16.h>

#include "tv_internal.h"

namespace {

constexpr int kConvThreads = 256;
constexpr int kConvWarps = kConvThreads / 32;
constexpr int kMaxConvDim = 256;

struct ConvArgs {
  const int32_t* parent;  // [n_trees][T]
  int32_t n_trees;
  int32_t B, H, T, dk, dv, W, normalize;
  float eps;
  const void* x;      // [B][T][C]
  const void* ctx;    // [B][W-1][C]
  const float* weight;  // [C][W]
  const float* bias;    // [C] or null
  const void* gate_a;   // [B][T][H] or null
  const void* gate_b;   // [B][T][H] or null
  const float* A_log;
  const float* dt_bias;
  void* q;
  void* k;
  void* v;
  float* alpha;
  float* beta;
};

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

// For memory the same kernel also writes (the in-place context commit): a coherent load that the
// compiler may not reorder against the stores.
__device__ __forceinline__ uint4 ld_ordered16(const void* p) {
  uint4 r;
  asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p)
               : "memory");
  return r;
}

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

// four consecutive channels of one staged row
__device__ __forceinline__ void load4(const float* row, int c, float (&o)[4]) {
  const float4 t = *reinterpret_cast<const float4*>(row + c);
  o[0] = t.x; o[1] = t.y; o[2] = t.z; o[3] = t.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* row, int c, float (&o)[4]) {
  const uint2 t = *reinterpret_cast<const uint2*>(row + c);
  o[0] = __uint_as_float(t.x << 16);
  o[1] = __uint_as_float(t.x & 0xffff0000u);
  o[2] = __uint_as_float(t.y << 16);
  o[3] = __uint_as_float(t.y & 0xffff0000u);
}
__device__ __forceinline__ void store4(float* dst, const float (&y)[4]) {
  asm volatile("st.global.L1::no_allocate.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(dst), "f"(y[0]),
               "f"(y[1]), "f"(y[2]), "f"(y[3])
               : "memory");
}
__device__ __forceinline__ void store4(__nv_bfloat16* dst, const float (&y)[4]) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(y[0], y[1]);
  const __nv_bfloat162 hi = __floats2bfloat162_rn(y[2], y[3]);
  asm volatile("st.global.L1::no_allocate.v2.u32 [%0], {%1,%2};" ::"l"(dst),
               "r"(*reinterpret_cast<const uint32_t*>(&lo)),
               "r"(*reinterpret_cast<const uint32_t*>(&hi))
               : "memory");
}

// SiLU(z) = z / (1 + e^-z).  e^-z overflows to +inf for z < -88 and the quotient is then -0.
__device__ __forceinline__ float silu(float z) { return __fdividef(z, 1.0f + __expf(-z)); }

__device__ __forceinline__ float softplus(float z) {
  return fmaxf(z, 0.0f) + log1pf(expf(-fabsf(z)));
}

// Shared memory: [T+W-1][d] staged rows (context rows first, oldest first, then the nodes),
// then the parent array, then 8 tap-row bytes per node.
template <typename IO, int W, int NJ>
__global__ void __launch_bounds__(kConvThreads)
tree_conv_kernel(const ConvArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int VEC = 16 / (int)sizeof(IO);
  const int T = a.T, H = a.H;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int slice = blockIdx.x % (3 * H), b = blockIdx.x / (3 * H);
  const int kind = slice / H, h = slice - kind * H;  // 0 q, 1 k, 2 v
  const int d = kind == 2 ? a.dv : a.dk;
  const int C = H * (2 * a.dk + a.dv);
  const int c0 = kind == 0 ? h * a.dk : kind == 1 ? (H + h) * a.dk : 2 * H * a.dk + h * a.dv;
  const int dmax = a.dk > a.dv ? a.dk : a.dv;
  const int rows = T + W - 1;

  IO* xs = reinterpret_cast<IO*>(smem_raw);
  int32_t* par_s = reinterpret_cast<int32_t*>(smem_raw + (size_t)(T + W - 1) * dmax * sizeof(IO));
  unsigned char* taps_s = reinterpret_cast<unsigned char*>(par_s + ((T + 1) & ~1));

  if (tid < T) par_s[tid] = a.parent[(size_t)(a.n_trees == 1 ? 0 : b) * T + tid];

  // ---- stage the slice: all loads of a batch are issued before the first store
  {
    const int vpr = d / VEC, total = rows * vpr;
    const IO* xb = reinterpret_cast<const IO*>(a.x) + (size_t)b * T * C + c0;
    const IO* cb = reinterpret_cast<const IO*>(a.ctx) + (size_t)b * (W - 1) * C + c0;
    for (int base = 0; base < total; base += 4 * kConvThreads) {
      uint4 r[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int idx = base + u * kConvThreads + tid;
        if (idx < total) {
          const int row = idx / vpr, col = (idx - row * vpr) * VEC;
          const IO* src = row < W - 1 ? cb + (size_t)row * C + col : xb + (size_t)(row - (W - 1)) * C + col;
          r[u] = ld_stream16(src);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int idx = base + u * kConvThreads + tid;
        if (idx < total) {
          const int row = idx / vpr, col = (idx - row * vpr) * VEC;
          *reinterpret_cast<uint4*>(xs + (size_t)row * d + col) = r[u];
        }
      }
    }
  }

  // ---- this lane's filter taps and bias: channels 4*lane + 128*j
  float wreg[NJ][W][4], breg[NJ][4];
#pragma unroll
  for (int j = 0; j < NJ; ++j) {
    const int c = 4 * lane + 128 * j;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const bool live = c + e < d;
      breg[j][e] = live && a.bias ? __ldg(a.bias + c0 + c + e) : 0.0f;
#pragma unroll
      for (int r = 0; r < W; ++r)
        wreg[j][r][e] = live ? __ldg(a.weight + (size_t)(c0 + c + e) * W + (W - 1 - r)) : 0.0f;
    }
  }

  // ---- gate preparation for this (request, head): done by the q slice
  if (kind == 0 && a.gate_a != nullptr && tid < T) {
    const size_t gi = ((size_t)b * T + tid) * H + h, go = ((size_t)b * H + h) * T + tid;
    const float ga = to_f32(reinterpret_cast<const IO*>(a.gate_a)[gi]);
    a.alpha[go] = expf(-expf(__ldg(a.A_log + h)) * softplus(ga + __ldg(a.dt_bias + h)));
    if (a.gate_b != nullptr) {
      const float gb = to_f32(reinterpret_cast<const IO*>(a.gate_b)[gi]);
      a.beta[go] = 1.0f / (1.0f + expf(-gb));
    }
  }
  __syncthreads();

  // ---- tap rows of every node: itself, its ancestors, then the context from its newest row
  if (tid < T) {
    int j = tid, ctx_row = W - 2;
#pragma unroll
    for (int r = 0; r < W; ++r) {
      int row;
      if (j >= 0) {
        row = W - 1 + j;
        j = par_s[j];
      } else {
        row = ctx_row--;
      }
      taps_s[tid * 8 + r] = (unsigned char)row;
    }
  }
  __syncthreads();

  // ---- one warp per node row
  IO* out = reinterpret_cast<IO*>(kind == 0 ? a.q : kind == 1 ? a.k : a.v) + ((size_t)b * H + h) * T * d;
  const bool norm = a.normalize && kind < 2;
#pragma unroll 2
  for (int i = warp; i < T; i += kConvWarps) {
    const uint2 tw = *reinterpret_cast<const uint2*>(taps_s + i * 8);
    float y[NJ][4];
    float ss = 0.0f;
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
      const int c = 4 * lane + 128 * j;
#pragma unroll
      for (int e = 0; e < 4; ++e) y[j][e] = breg[j][e];
      if (c < d) {
#pragma unroll
        for (int r = 0; r < W; ++r) {
          const uint32_t row = ((r < 4 ? tw.x : tw.y) >> (8 * (r & 3))) & 0xffu;
          float in[4];
          load4(xs + (size_t)row * d, c, in);
#pragma unroll
          for (int e = 0; e < 4; ++e) y[j][e] = fmaf(wreg[j][r][e], in[e], y[j][e]);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          y[j][e] = silu(y[j][e]);
          ss = fmaf(y[j][e], y[j][e], ss);
        }
      }
    }
    if (norm) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      const float sc = 1.0f / sqrtf(ss + a.eps);
#pragma unroll
      for (int j = 0; j < NJ; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) y[j][e] *= sc;
    }
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
      const int c = 4 * lane + 128 * j;
      if (c < d) store4(out + (size_t)i * d + c, y[j]);
    }
  }
}

// Context rows after the commit: one thread per 16-byte channel vector reads its W-1 source
// values (accepted node and its ancestors first, then the old context) before it writes any, so
// ctx_new may be ctx itself.
template <typename IO, int W>
__global__ void __launch_bounds__(kConvThreads)
conv_commit_kernel(const int32_t* __restrict__ parent, int32_t n_trees, const int32_t* __restrict__ accepted,
                   int32_t T, int32_t C, const IO* x, const IO* ctx, IO* ctx_new) {
  constexpr int VEC = 16 / (int)sizeof(IO);
  const int b = blockIdx.y;
  const int col = (blockIdx.x * kConvThreads + threadIdx.x) * VEC;
  if (col >= C) return;
  int acc = accepted[b];
  if (acc >= T) acc = -1;
  const int32_t* par = parent + (size_t)(n_trees == 1 ? 0 : b) * T;
  const IO* xb = x + (size_t)b * T * C + col;
  const IO* cb = ctx + (size_t)b * (W - 1) * C + col;
  uint4 vals[W > 1 ? W - 1 : 1];
  int j = acc, back = W - 2;
#pragma unroll
  for (int t = 0; t < W - 1; ++t) {  // t = 0 is the newest row
    if (j >= 0) {
      vals[t] = ld_ordered16(xb + (size_t)j * C);
      j = __ldg(par + j);
    } else {
      vals[t] = ld_ordered16(cb + (size_t)(back--) * C);
    }
  }
  IO* ob = ctx_new + (size_t)b * (W - 1) * C + col;
#pragma unroll
  for (int t = 0; t < W - 1; ++t) *reinterpret_cast<uint4*>(ob + (size_t)(W - 2 - t) * C) = vals[t];
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

int check_conv(const tv_tree* t, const tv_conv_dims* d) {
  if (!t || !d) return TV_ERR_BAD_ARG;
  if (d->B < 1 || d->H < 1 || d->T < 1 || d->dk < 1 || d->dv < 1 || d->W < 1) return TV_ERR_BAD_ARG;
  if (d->io_dtype != TV_F32 && d->io_dtype != TV_BF16) return TV_ERR_BAD_ARG;
  if (d->T > TV_MAX_NODES || d->dk > kMaxConvDim || d->dv > kMaxConvDim || d->W > TV_CONV_MAX_TAPS)
    return TV_ERR_UNSUPPORTED;
  const int m = d->io_dtype == TV_BF16 ? 7 : 3;
  if ((d->dk & m) || (d->dv & m)) return TV_ERR_UNSUPPORTED;
  if (t->n != d->T) return TV_ERR_BAD_ARG;
  if (t->n_trees != 1 && t->n_trees != d->B) return TV_ERR_BAD_ARG;
  if ((int64_t)d->B * d->H * 3 > 0x7fffffffLL || d->B > 65535) return TV_ERR_UNSUPPORTED;
  if (!t->uploaded) return TV_ERR_NOT_UPLOADED;
  return TV_OK;
}

template <typename IO, int W>
int launch_conv(const ConvArgs& a, cudaStream_t stream) {
  const int dmax = a.dk > a.dv ? a.dk : a.dv;
  const size_t smem = (size_t)(a.T + W - 1) * dmax * sizeof(IO) + (size_t)((a.T + 1) & ~1) * 4 + (size_t)a.T * 8;
  const unsigned grid = (unsigned)a.B * 3u * (unsigned)a.H;
  auto go = [&](auto kernel) -> int {
    if (smem > 48 * 1024)
      TV_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kernel<<<grid, kConvThreads, smem, stream>>>(a);
    TV_CUDA_TRY(cudaGetLastError());
    return TV_OK;
  };
  return dmax <= 128 ? go(tree_conv_kernel<IO, W, 1>) : go(tree_conv_kernel<IO, W, 2>);
}

template <typename IO>
int launch_conv_w(const ConvArgs& a, cudaStream_t s) {
  switch (a.W) {
    case 1: return launch_conv<IO, 1>(a, s);
    case 2: return launch_conv<IO, 2>(a, s);
    case 3: return launch_conv<IO, 3>(a, s);
    case 4: return launch_conv<IO, 4>(a, s);
    case 5: return launch_conv<IO, 5>(a, s);
    case 6: return launch_conv<IO, 6>(a, s);
    case 7: return launch_conv<IO, 7>(a, s);
    case 8: return launch_conv<IO, 8>(a, s);
  }
  return TV_ERR_UNSUPPORTED;
}

template <typename IO, int W>
int launch_conv_commit(const tv_tree* t, const tv_conv_dims* d, const int32_t* accepted, const void* x,
                       const void* ctx, void* ctx_new, cudaStream_t s) {
  constexpr int VEC = 16 / (int)sizeof(IO);
  const int C = d->H * (2 * d->dk + d->dv);
  dim3 grid((unsigned)((C / VEC + kConvThreads - 1) / kConvThreads), (unsigned)d->B);
  conv_commit_kernel<IO, W><<<grid, kConvThreads, 0, s>>>(t->d_parent, t->n_trees, accepted, d->T, C,
                                                         (const IO*)x, (const IO*)ctx, (IO*)ctx_new);
  TV_CUDA_TRY(cudaGetLastError());
  return TV_OK;
}

template <typename IO>
int launch_conv_commit_w(const tv_tree* t, const tv_conv_dims* d, const int32_t* acc, const void* x,
                         const void* ctx, void* ctx_new, cudaStream_t s) {
  switch (d->W) {
    case 2: return launch_conv_commit<IO, 2>(t, d, acc, x, ctx, ctx_new, s);
    case 3: return launch_conv_commit<IO, 3>(t, d, acc, x, ctx, ctx_new, s);
    case 4: return launch_conv_commit<IO, 4>(t, d, acc, x, ctx, ctx_new, s);
    case 5: return launch_conv_commit<IO, 5>(t, d, acc, x, ctx, ctx_new, s);
    case 6: return launch_conv_commit<IO, 6>(t, d, acc, x, ctx, ctx_new, s);
    case 7: return launch_conv_commit<IO, 7>(t, d, acc, x, ctx, ctx_new, s);
    case 8: return launch_conv_commit<IO, 8>(t, d, acc, x, ctx, ctx_new, s);
  }
  return TV_ERR_UNSUPPORTED;
}

}  // namespace

#define TV_API __attribute__((visibility("default")))

extern "C" {

TV_API int tv_tree_conv(const tv_tree* tree, const tv_conv_dims* d, const void* x, const void* ctx,
                        const float* weight, const float* bias, const void* gate_a, const void* gate_b,
                        const float* A_log, const float* dt_bias, void* q, void* k, void* v,
                        float* alpha, float* beta, void* stream) {
  int st = check_conv(tree, d);
  if (st != TV_OK) return st;
  if (!x || !weight || !q || !k || !v) return TV_ERR_BAD_ARG;
  if (d->W > 1 && !ctx) return TV_ERR_BAD_ARG;
  if (gate_a && (!A_log || !dt_bias || !alpha)) return TV_ERR_BAD_ARG;
  if (gate_b && (!gate_a || !beta)) return TV_ERR_BAD_ARG;
  if (!aligned16(x) || !aligned16(ctx) || !aligned16(q) || !aligned16(k) || !aligned16(v) ||
      ((uintptr_t)weight & 3) || ((uintptr_t)bias & 3) || ((uintptr_t)alpha & 3) || ((uintptr_t)beta & 3) ||
      ((uintptr_t)A_log & 3) || ((uintptr_t)dt_bias & 3))
    return TV_ERR_BAD_ARG;
  const uintptr_t esz = d->io_dtype == TV_BF16 ? 2 : 4;
  if (((uintptr_t)gate_a & (esz - 1)) || ((uintptr_t)gate_b & (esz - 1))) return TV_ERR_BAD_ARG;
  if (q == x || k == x || v == x || q == k || q == v || k == v) return TV_ERR_BAD_ARG;
  ConvArgs a;
  a.parent = tree->d_parent; a.n_trees = tree->n_trees;
  a.B = d->B; a.H = d->H; a.T = d->T; a.dk = d->dk; a.dv = d->dv; a.W = d->W;
  a.normalize = d->normalize_qk != 0; a.eps = d->eps;
  a.x = x; a.ctx = ctx; a.weight = weight; a.bias = bias; a.gate_a = gate_a; a.gate_b = gate_b;
  a.A_log = A_log; a.dt_bias = dt_bias; a.q = q; a.k = k; a.v = v; a.alpha = alpha; a.beta = beta;
  return d->io_dtype == TV_BF16 ? launch_conv_w<__nv_bfloat16>(a, (cudaStream_t)stream)
                                : launch_conv_w<float>(a, (cudaStream_t)stream);
}

TV_API int tv_conv_commit(const tv_tree* tree, const tv_conv_dims* d, const int32_t* accepted,
                          const void* x, const void* ctx, void* ctx_new, void* stream) {
  int st = check_conv(tree, d);
  if (st != TV_OK) return st;
  if (d->W == 1) return TV_OK;  // no context to keep
  if (!accepted || !x || !ctx || !ctx_new) return TV_ERR_BAD_ARG;
  if (!aligned16(x) || !aligned16(ctx) || !aligned16(ctx_new) || ((uintptr_t)accepted & 3)) return TV_ERR_BAD_ARG;
  if (ctx_new != ctx) {
    const size_t esz = d->io_dtype == TV_BF16 ? 2 : 4;
    const size_t bytes = esz * (size_t)d->B * (d->W - 1) * d->H * (2 * d->dk + d->dv);
    const char* a0 = (const char*)ctx;
    const char* b0 = (const char*)ctx_new;
    if (a0 < b0 + bytes && b0 < a0 + bytes) return TV_ERR_BAD_ARG;  // partial overlap
  }
  if (ctx_new == x) return TV_ERR_BAD_ARG;
  return d->io_dtype == TV_BF16
             ? launch_conv_commit_w<__nv_bfloat16>(tree, d, accepted, x, ctx, ctx_new, (cudaStream_t)stream)
             : launch_conv_commit_w<float>(tree, d, accepted, x, ctx, ctx_new, (cudaStream_t)stream);
}

}  // extern "C"
