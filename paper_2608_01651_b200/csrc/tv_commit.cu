// Accepted-path commit (Section IV-D Eq. 10; Lemma 1 Eq. 3).
//
//   S_new[v][k] = P_a S_pre[v][k] + sum_{j in P(a)} (P_a/P_j) u_j[v] k_j[k]
//
// One CTA streams one (layer, request, head) state of dv x dk floats through
// registers exactly once: 16-byte loads issued back to back, the rank-len
// update applied from shared memory, 16-byte stores.  HBM-bound: 8 dk dv bytes
// per state against (1 + len) FMAs per element.
//
// The accepted path needs no parent walk: node indices grow along a
// root-to-node path, so the set bits of the 128-bit ancestor mask of a, plus a
// itself, are the path in topological order.
//
// Every kernel takes its tensors layer by layer from a table in its parameters (Section IV-D /
// V-B: all linear layers are committed by one launch, whether they are stacked in one allocation
// or own their caches separately); work item -> (layer, request, head), tensors of that layer,
// rows addressed through the layout's strides within the layer.
#include <cuda_bf16.h>

#include "tv_internal.h"

namespace {

constexpr int kThreads = 256;
constexpr int kPathChunk = 16;  // path rows staged in shared memory at a time
constexpr int kMaxVec = 16;     // float4 per thread: dk*dv <= 16384

template <bool BF16>
__device__ __forceinline__ float load_elem(const void* base, size_t idx) {
  if (BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(base)[idx]);
  return reinterpret_cast<const float*>(base)[idx];
}

// Work item -> layer and item within the layer.
struct LayerItem {
  int l, it;   // layer of this launch, (request, head) item inside the layer
  int b;       // request
};
__device__ __forceinline__ LayerItem layer_item(const CommitArgs& a, int item) {
  LayerItem r;
  const int bh = a.B * a.H;
  r.l = item / bh;
  r.it = item - r.l * bh;
  r.b = r.it / a.H;
  return r;
}
__device__ __forceinline__ ItemRows rows_of(const CommitArgs& a, int it_in_layer) {
  return tv_item_rows(a.tree, a.lay, it_in_layer, a.B, a.H, a.Hk, a.T, a.dk, a.dv);
}

// Fills path_s[0..len) (topological order), w_s[p] = P_a / P_path[p] and *Pa_s.
// al_s is scratch for the T decay gates (loaded by T threads in parallel so that
// the serial suffix product below never waits on global memory).
__device__ __forceinline__ int build_path(const TreeDev& tree, size_t meta0, int T, int acc,
                                          const float* alpha, size_t g0, int64_t g_rs, int* path_s, float* w_s,
                                          float* al_s, float* Pa_s) {
  const uint64_t* m = tree.anc + (meta0 + acc) * 2;
  const int t = threadIdx.x;
  if (t < T) al_s[t] = alpha[g0 + (size_t)t * g_rs];
  uint64_t m0 = m[0], m1 = m[1];
  if (acc < 64) m0 |= 1ull << acc; else m1 |= 1ull << (acc - 64);
  const int len = __popcll(m0) + __popcll(m1);
  if (t < 128) {
    const uint64_t w = t < 64 ? m0 : m1;
    const int bit = t & 63;
    if ((w >> bit) & 1) {
      int pos = __popcll(w & ((1ull << bit) - 1));
      if (t >= 64) pos += __popcll(m0);
      path_s[pos] = t;
    }
  }
  __syncthreads();
  if (t == 0) {
    float w = 1.f;
    for (int p = len - 1; p >= 0; --p) {
      w_s[p] = w;
      w *= al_s[path_s[p]];
    }
    *Pa_s = w;
  }
  __syncthreads();
  return len;
}

// Streaming 16-byte load / store: the state is touched exactly once.
__device__ __forceinline__ float4 ld_stream(const float4* p) {
  float4 v;
  asm volatile("ld.global.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream(float4* p, const float4& v) {
  asm volatile("st.global.L1::no_allocate.v4.f32 [%0], {%1,%2,%3,%4};"
               :: "l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}

// Commit from given correction rows u_j: U (float) when given, else v.
template <bool BF16>
__global__ void __launch_bounds__(kThreads)
commit_factored_kernel(const CommitArgs a, const __grid_constant__ CommitLayers tb) {
  asm volatile("griddepcontrol.wait;" ::: "memory");   // dependent launch: nothing is read before the kernel in front is done
  __shared__ int path_s[TV_MAX_NODES];
  __shared__ float w_s[TV_MAX_NODES];
  __shared__ float Pa_s;
  __shared__ float al_s[TV_MAX_NODES];
  __shared__ __align__(16) float k_s[kPathChunk][TV_MAX_DIM];
  __shared__ float cu_s[kPathChunk][TV_MAX_DIM];

  const LayerItem li = layer_item(a, blockIdx.x);
  const int tid = threadIdx.x;
  const int dk = a.dk, dv = a.dv;
  const ItemRows rows = rows_of(a, li.it);
  const int T = rows.n;
  const int n4 = dv * dk / 4;
  const size_t sbase = (size_t)li.it * dv * dk;
  const float4* src = reinterpret_cast<const float4*>(tb.S_pre[li.l] + sbase);
  float4* dst = reinterpret_cast<float4*>(tb.S_new[li.l] + sbase);
  const void* kg = tb.k[li.l];
  const void* vg = tb.v[li.l];
  const float* Ug = tb.U[li.l];

  int acc = a.accepted[li.b];
  if (acc >= T) acc = -1;
  if (acc < 0) {
    if (!a.in_place)
      for (int i = tid; i < n4; i += kThreads) st_stream(dst + i, ld_stream(src + i));
    return;
  }
  // The whole state goes in flight first; the path is worked out under its latency.
  float4 s[kMaxVec];
#pragma unroll
  for (int e = 0; e < kMaxVec; ++e) {
    const int i = tid + e * kThreads;
    if (i < n4) s[e] = ld_stream(src + i);
  }
  const int len = build_path(a.tree, rows.meta0, T, acc, tb.alpha[li.l], rows.g0, rows.g_rs, path_s, w_s, al_s, &Pa_s);
  const float Pa = Pa_s;
#pragma unroll
  for (int e = 0; e < kMaxVec; ++e) {
    s[e].x *= Pa; s[e].y *= Pa; s[e].z *= Pa; s[e].w *= Pa;
  }
  const int dk4 = dk >> 2;
  for (int c0 = 0; c0 < len; c0 += kPathChunk) {
    const int nc = min(kPathChunk, len - c0);
    __syncthreads();
    for (int i = tid; i < nc * dk; i += kThreads) {
      const int p = i / dk, kk = i - p * dk;
      k_s[p][kk] = load_elem<BF16>(kg, rows.qk0 + (size_t)path_s[c0 + p] * rows.qk_rs + kk);
    }
    for (int i = tid; i < nc * dv; i += kThreads) {
      const int p = i / dv, vv = i - p * dv;
      const float u = a.has_U ? Ug[rows.o0 + (size_t)path_s[c0 + p] * rows.o_rs + vv]
                              : load_elem<BF16>(vg, rows.v0 + (size_t)path_s[c0 + p] * rows.v_rs + vv);
      cu_s[p][vv] = w_s[c0 + p] * u;
    }
    __syncthreads();
#pragma unroll
    for (int e = 0; e < kMaxVec; ++e) {
      const int i = tid + e * kThreads;
      if (i < n4) {
        const int row = i / dk4, c4 = i - row * dk4;
        for (int p = 0; p < nc; ++p) {
          const float cu = cu_s[p][row];
          const float4 kv = *reinterpret_cast<const float4*>(&k_s[p][c4 * 4]);
          s[e].x = fmaf(cu, kv.x, s[e].x);
          s[e].y = fmaf(cu, kv.y, s[e].y);
          s[e].z = fmaf(cu, kv.z, s[e].z);
          s[e].w = fmaf(cu, kv.w, s[e].w);
        }
      }
    }
  }
#pragma unroll
  for (int e = 0; e < kMaxVec; ++e) {
    const int i = tid + e * kThreads;
    if (i < n4) st_stream(dst + i, s[e]);
  }
}

// dk = 128 fast path.  A CTA of 4 warps owns 64 consecutive rows (value
// channels) of one state; warp w owns rows 16w..16w+15 and a lane owns one
// float4 column, so every load and store of a warp is one contiguous 512-byte
// row and the key row k_j[4 lane .. 4 lane + 3] stays in registers across the
// 16 rows.  All 16 loads of a thread are in flight before anything else
// happens; several CTAs per SM keep the stream continuous.
constexpr int kRowThreads = 128;
constexpr int kRowsPerCta = 64;

// Four keys of a path row, widened to float.
template <bool BF16>
__device__ __forceinline__ float4 load_key4(const void* kg, size_t idx) {
  if (BF16) {
    const uint2 r = *reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(kg) + idx);
    return make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xffff0000u),
                       __uint_as_float(r.y << 16), __uint_as_float(r.y & 0xffff0000u));
  }
  return *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(kg) + idx);
}

template <bool BF16>
__global__ void __launch_bounds__(kRowThreads)
commit_factored_dk128_kernel(const CommitArgs a, const __grid_constant__ CommitLayers tb) {
  __shared__ int path_s[TV_MAX_NODES];
  __shared__ float w_s[TV_MAX_NODES];
  __shared__ float Pa_s;
  __shared__ float al_s[TV_MAX_NODES];
  __shared__ __align__(16) float k_s[kPathChunk][128];
  __shared__ __align__(16) float cu_s[kPathChunk][kRowsPerCta];

  const int dv = a.dv;
  const int n_half = (dv + kRowsPerCta - 1) / kRowsPerCta;
  const int item = blockIdx.x / n_half, half = blockIdx.x - item * n_half;
  const LayerItem li = layer_item(a, item);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row0 = half * kRowsPerCta + warp * 16;
  const size_t sbase = (size_t)li.it * dv * 128;
  const float4* src = reinterpret_cast<const float4*>(tb.S_pre[li.l] + sbase) + (size_t)row0 * 32 + lane;
  float4* dst = reinterpret_cast<float4*>(tb.S_new[li.l] + sbase) + (size_t)row0 * 32 + lane;

  int acc = a.accepted[li.b];
  if (acc >= a.T) acc = -1;
  if (acc < 0 && a.in_place) return;
  float4 s[16];
#pragma unroll
  for (int e = 0; e < 16; ++e)
    if (row0 + e < dv) s[e] = ld_stream(src + e * 32);
  // Dependent launch: this grid may have started under the tail of the kernel in front of it
  // (a verify kernel, or the tree-metadata kernel when no verify call sits in between).  S_pre
  // and the accepted nodes are older than either; everything those kernels write -- U, and the
  // tree metadata including the request offsets of a packed forest -- is read, and everything
  // they read that we write (S in place) is written, after this point.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const ItemRows rows = rows_of(a, li.it);
  const int T = rows.n;
  if (acc >= T) acc = -1;   // packed forest: beyond this request's node count
  if (acc < 0) {
    if (a.in_place) return;
#pragma unroll
    for (int e = 0; e < 16; ++e)
      if (row0 + e < dv) st_stream(dst + e * 32, s[e]);
    return;
  }
  const void* kg = tb.k[li.l];
  const void* vg = tb.v[li.l];
  const float* Ug = tb.U[li.l];
  const int len = build_path(a.tree, rows.meta0, T, acc, tb.alpha[li.l], rows.g0, rows.g_rs, path_s, w_s, al_s, &Pa_s);
  const float Pa = Pa_s;
  bool scaled = false;
  for (int c0 = 0; c0 < len; c0 += kPathChunk) {
    const int nc = min(kPathChunk, len - c0);
    if (c0) __syncthreads();
    for (int i = tid; i < nc * 32; i += kRowThreads) {   // 4 keys per thread per step
      const int p = i >> 5, k4 = i & 31;
      *reinterpret_cast<float4*>(&k_s[p][k4 * 4]) =
          load_key4<BF16>(kg, rows.qk0 + (size_t)path_s[c0 + p] * rows.qk_rs + k4 * 4);
    }
    for (int i = tid; i < nc * kRowsPerCta; i += kRowThreads) {
      const int p = i >> 6, r = i & 63;
      const int vrow = half * kRowsPerCta + r;
      float u = 0.f;
      if (vrow < dv)
        u = a.has_U ? Ug[rows.o0 + (size_t)path_s[c0 + p] * rows.o_rs + vrow]
                    : load_elem<BF16>(vg, rows.v0 + (size_t)path_s[c0 + p] * rows.v_rs + vrow);
      cu_s[p][r] = w_s[c0 + p] * u;
    }
    __syncthreads();
    if (!scaled) {   // first use of the state: the loads have had the path build to land
      scaled = true;
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        s[e].x *= Pa; s[e].y *= Pa; s[e].z *= Pa; s[e].w *= Pa;
      }
    }
    for (int p = 0; p < nc; ++p) {
      const float4 kv = *reinterpret_cast<const float4*>(&k_s[p][lane * 4]);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float4 cu = *reinterpret_cast<const float4*>(&cu_s[p][warp * 16 + q * 4]);
        const float c[4] = {cu.x, cu.y, cu.z, cu.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          float4& x = s[q * 4 + t];
          x.x = fmaf(c[t], kv.x, x.x);
          x.y = fmaf(c[t], kv.y, x.y);
          x.z = fmaf(c[t], kv.z, x.z);
          x.w = fmaf(c[t], kv.w, x.w);
        }
      }
    }
  }
#pragma unroll
  for (int e = 0; e < 16; ++e) {
    if (row0 + e < dv) st_stream(dst + e * 32, s[e]);
  }
}

// Persistent version of the dk = 128 row-owner kernel for accepted paths of at most 16 nodes
// and batches of at most 256 requests.  A CTA walks units of 64 state rows; the accepted node
// and path mask of every request are read once per CTA, and while the 16 loads of unit n are
// in flight the path of unit n+1 is worked out (nodes from the mask bits, suffix products
// P_a/P_j by a warp scan) and its key / value rows are fetched into registers, to be staged in
// the other half of a double buffer after unit n has been updated.  No unit waits on a chain of
// dependent global loads.
#ifndef TV_STREAM_CTAS
#define TV_STREAM_CTAS 5
#endif
constexpr int kStreamMaxB = 256;
constexpr int kStreamMaxLen = 16;

template <bool BF16>
__global__ void __launch_bounds__(kRowThreads, TV_STREAM_CTAS)
commit_stream_dk128_kernel(const CommitArgs a, const __grid_constant__ CommitLayers tb) {
  __shared__ int acc_s[kStreamMaxB];
  __shared__ uint64_t mask_s[kStreamMaxB][2];
  __shared__ __align__(16) float k_s[2][kStreamMaxLen][128];
  __shared__ __align__(16) float cu_s[2][kStreamMaxLen][kRowsPerCta];
  __shared__ int node_s[2][kStreamMaxLen];
  __shared__ float w_s[2][kStreamMaxLen];
  __shared__ float Pa_s[2];
  __shared__ int len_s[2];

  const int dv = a.dv, T = a.T;
  const int n_half = dv / kRowsPerCta;
  const int n_units = a.L * a.B * a.H * n_half;
  const int units_per_layer = a.B * a.H * n_half;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool in_place = a.in_place != 0;

  for (int b = tid; b < a.B; b += kRowThreads) {
    int acc = a.accepted[b];
    const int nb = a.tree.offsets ? a.tree.offsets[b + 1] - a.tree.offsets[b] : T;
    if (acc >= nb) acc = -1;
    acc_s[b] = acc;
    uint64_t m0 = 0, m1 = 0;
    if (acc >= 0) {
      const int tb_ = a.tree.n_trees == 1 ? 0 : b;
      const uint64_t* m = a.tree.anc + ((size_t)tb_ * T + acc) * 2;
      m0 = m[0];
      m1 = m[1];
      if (acc < 64) m0 |= 1ull << acc; else m1 |= 1ull << (acc - 64);
    }
    mask_s[b][0] = m0;
    mask_s[b][1] = m1;
  }
  __syncthreads();

  auto req_of = [&](int u) { return ((u / n_half) / a.H) % a.B; };
  auto next_live = [&](int u) {   // first unit >= u (in this CTA's stride) that has work to do
    while (u < n_units && in_place && acc_s[req_of(u)] < 0) u += gridDim.x;
    return u;
  };

  // path of unit u into buffer nb: nodes, weights P_a/P_j, P_a, length (warp 0)
  auto path_nodes = [&](int u, int nb) {
    if (warp != 0) return;
    const int b = req_of(u);
    const uint64_t m0 = mask_s[b][0], m1 = mask_s[b][1];
    const int c0 = __popcll(m0);
    const int len = min(c0 + __popcll(m1), kStreamMaxLen);
    int node = 0;
    float al = 1.f;
    if (lane < len) {
      uint64_t w = lane < c0 ? m0 : m1;
      const int r = lane < c0 ? lane : lane - c0;
      for (int i = 0; i < r; ++i) w &= w - 1;
      node = __ffsll((long long)w) - 1 + (lane < c0 ? 0 : 64);
      const LayerItem li = layer_item(a, u / n_half);
      const ItemRows rows = rows_of(a, li.it);
      al = tb.alpha[li.l][rows.g0 + (size_t)node * rows.g_rs];
    }
    float incl = al;   // product of alpha over path positions >= lane
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const float up = __shfl_down_sync(0xffffffffu, incl, o);
      if (lane + o < 32) incl *= up;
    }
    const float nxt = __shfl_down_sync(0xffffffffu, incl, 1);
    if (lane < kStreamMaxLen) {
      node_s[nb][lane] = node;
      w_s[nb][lane] = lane + 1 < 32 ? nxt : 1.f;
    }
    if (lane == 0) {
      Pa_s[nb] = incl;
      len_s[nb] = len;
    }
  };

  // key / value rows of unit u's path: 4 x 16 keys and 8 values per thread, in registers
  uint2 kreg[4];
  uint2 kreg2[4];
  float ureg[8];
  auto fetch_rows = [&](int u, int nb) {
    const int item = u / n_half, half = u - item * n_half;
    const LayerItem li = layer_item(a, item);
    const ItemRows rows = rows_of(a, li.it);
    const void* kg = tb.k[li.l];
    const void* vg = tb.v[li.l];
    const float* Ug = tb.U[li.l];
    const int len = len_s[nb];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int i = tid + q * kRowThreads;          // (p, k4) = (i / 32, i % 32)
      const int p = i >> 5, k4 = i & 31;
      kreg[q] = make_uint2(0u, 0u);
      kreg2[q] = make_uint2(0u, 0u);
      if (p < len) {
        const size_t idx = rows.qk0 + (size_t)node_s[nb][p] * rows.qk_rs + k4 * 4;
        if (BF16) {
          kreg[q] = *reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(kg) + idx);
        } else {
          const uint4 r = *reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(kg) + idx);
          kreg[q] = make_uint2(r.x, r.y);
          kreg2[q] = make_uint2(r.z, r.w);
        }
      }
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int i = tid + q * kRowThreads;          // (p, r) = (i / 64, i % 64)
      const int p = i >> 6, r = i & 63;
      ureg[q] = 0.f;
      if (p < len) {
        const int vrow = half * kRowsPerCta + r;
        ureg[q] = a.has_U ? Ug[rows.o0 + (size_t)node_s[nb][p] * rows.o_rs + vrow]
                          : load_elem<BF16>(vg, rows.v0 + (size_t)node_s[nb][p] * rows.v_rs + vrow);
      }
    }
  };
  auto stage_rows = [&](int nb) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int i = tid + q * kRowThreads;
      const int p = i >> 5, k4 = i & 31;
      float4 kv;
      if (BF16) {
        kv = make_float4(__uint_as_float(kreg[q].x << 16), __uint_as_float(kreg[q].x & 0xffff0000u),
                         __uint_as_float(kreg[q].y << 16), __uint_as_float(kreg[q].y & 0xffff0000u));
      } else {
        kv = make_float4(__uint_as_float(kreg[q].x), __uint_as_float(kreg[q].y),
                         __uint_as_float(kreg2[q].x), __uint_as_float(kreg2[q].y));
      }
      *reinterpret_cast<float4*>(&k_s[nb][p][k4 * 4]) = kv;
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int i = tid + q * kRowThreads;
      const int p = i >> 6, r = i & 63;
      cu_s[nb][p][r] = w_s[nb][p] * ureg[q];
    }
  };

  int u = next_live(blockIdx.x);
  if (u >= n_units) return;
  path_nodes(u, 0);
  __syncthreads();
  fetch_rows(u, 0);
  stage_rows(0);
  __syncthreads();

  for (int n = 0; u < n_units; ++n) {
    const int cb = n & 1, nb = cb ^ 1;
    const int un = next_live(u + gridDim.x);
    // a. the 16 loads of this unit
    const int row0 = warp * 16;
    const int l = u / units_per_layer, ul = u - l * units_per_layer;
    const float4* src = reinterpret_cast<const float4*>(tb.S_pre[l]) + ((size_t)ul * kRowsPerCta + row0) * 32 + lane;
    float4* dst = reinterpret_cast<float4*>(tb.S_new[l]) + ((size_t)ul * kRowsPerCta + row0) * 32 + lane;
    float4 s[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) s[e] = ld_stream(src + e * 32);
    // b-d. the path of the next unit, and its rows into registers
    if (un < n_units) path_nodes(un, nb);
    __syncthreads();
    if (un < n_units) fetch_rows(un, nb);
    // e. update and store this unit
    const float Pa = Pa_s[cb];
    const int len = len_s[cb];
    if (len > 0) {
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        s[e].x *= Pa; s[e].y *= Pa; s[e].z *= Pa; s[e].w *= Pa;
      }
      for (int p = 0; p < len; ++p) {
        const float4 kv = *reinterpret_cast<const float4*>(&k_s[cb][p][lane * 4]);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 cu = *reinterpret_cast<const float4*>(&cu_s[cb][p][warp * 16 + q * 4]);
          const float c[4] = {cu.x, cu.y, cu.z, cu.w};
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            float4& x = s[q * 4 + t];
            x.x = fmaf(c[t], kv.x, x.x);
            x.y = fmaf(c[t], kv.y, x.y);
            x.z = fmaf(c[t], kv.z, x.z);
            x.w = fmaf(c[t], kv.w, x.w);
          }
        }
      }
    }
#pragma unroll
    for (int e = 0; e < 16; ++e) st_stream(dst + e * 32, s[e]);
    // f. the next unit's rows into the other buffer
    if (un < n_units) stage_rows(nb);
    __syncthreads();
    u = un;
  }
}

// Delta rule without stored corrections: every row v of the [dv][dk] state
// evolves independently along the accepted path,
//   s <- alpha_j s;  u = beta_j (v_j[v] - s . k_j);  s <- s + u k_j,
// which is the sequential rule restricted to one value channel.  A warp owns a
// row at a time (NPL consecutive floats per lane, dk = 32 NPL); the dot
// product is a shuffle reduction.
template <bool BF16, int NPL>
__global__ void __launch_bounds__(kThreads)
commit_delta_rows_kernel(const CommitArgs a, const __grid_constant__ CommitLayers tb) {
  asm volatile("griddepcontrol.wait;" ::: "memory");   // dependent launch: nothing is read before the kernel in front is done
  constexpr int DK = 32 * NPL;
  constexpr int kRowsPerWarp = TV_MAX_DIM / (kThreads / 32);  // 16
  __shared__ int path_s[TV_MAX_NODES];
  __shared__ float w_s[TV_MAX_NODES];
  __shared__ float Pa_s;
  __shared__ __align__(16) float k_s[kPathChunk][DK];
  __shared__ float v_s[kPathChunk][TV_MAX_DIM];
  __shared__ float alc_s[kPathChunk], be_s[kPathChunk];
  __shared__ float al_s[TV_MAX_NODES];

  const LayerItem li = layer_item(a, blockIdx.x);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int dv = a.dv;
  const ItemRows rows = rows_of(a, li.it);
  const int T = rows.n;
  const size_t sbase = (size_t)li.it * dv * DK;
  const int n4 = dv * DK / 4;
  const float* Sp = tb.S_pre[li.l] + sbase;
  float* Sn = tb.S_new[li.l] + sbase;
  const void* kg = tb.k[li.l];
  const void* vg = tb.v[li.l];
  const float* beta = tb.beta[li.l];

  int acc = a.accepted[li.b];
  if (acc >= T) acc = -1;
  if (acc < 0) {
    if (!a.in_place) {
      const float4* src = reinterpret_cast<const float4*>(Sp);
      float4* dst = reinterpret_cast<float4*>(Sn);
      for (int i = tid; i < n4; i += kThreads) dst[i] = src[i];
    }
    return;
  }
  const int len = build_path(a.tree, rows.meta0, T, acc, tb.alpha[li.l], rows.g0, rows.g_rs, path_s, w_s, al_s, &Pa_s);

  float s[kRowsPerWarp][NPL];
#pragma unroll
  for (int r = 0; r < kRowsPerWarp; ++r) {
    const int row = warp + r * (kThreads / 32);
    if (row < dv) {
      const float* p = Sp + (size_t)row * DK + lane * NPL;
      if (NPL == 4) {
        const float4 t = *reinterpret_cast<const float4*>(p);
        s[r][0] = t.x; s[r][1] = t.y; s[r][2 % NPL] = t.z; s[r][3 % NPL] = t.w;
      } else {
        const float2 t = *reinterpret_cast<const float2*>(p);
        s[r][0] = t.x; s[r][1] = t.y;
      }
    }
  }
  for (int c0 = 0; c0 < len; c0 += kPathChunk) {
    const int nc = min(kPathChunk, len - c0);
    __syncthreads();
    for (int i = tid; i < nc * DK; i += kThreads) {
      const int p = i / DK, kk = i - p * DK;
      k_s[p][kk] = load_elem<BF16>(kg, rows.qk0 + (size_t)path_s[c0 + p] * rows.qk_rs + kk);
    }
    for (int i = tid; i < nc * dv; i += kThreads) {
      const int p = i / dv, vv = i - p * dv;
      v_s[p][vv] = load_elem<BF16>(vg, rows.v0 + (size_t)path_s[c0 + p] * rows.v_rs + vv);
    }
    if (tid < nc) {
      alc_s[tid] = al_s[path_s[c0 + tid]];
      be_s[tid] = beta[rows.g0 + (size_t)path_s[c0 + tid] * rows.g_rs];
    }
    __syncthreads();
    for (int p = 0; p < nc; ++p) {
      float kr[NPL];
#pragma unroll
      for (int x = 0; x < NPL; ++x) kr[x] = k_s[p][lane * NPL + x];
      const float al = alc_s[p], be = be_s[p];
#pragma unroll
      for (int r = 0; r < kRowsPerWarp; ++r) {
        const int row = warp + r * (kThreads / 32);
        if (row < dv) {
          float dot = 0.f;
#pragma unroll
          for (int x = 0; x < NPL; ++x) {
            s[r][x] *= al;
            dot = fmaf(s[r][x], kr[x], dot);
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
          const float u = be * (v_s[p][row] - dot);
#pragma unroll
          for (int x = 0; x < NPL; ++x) s[r][x] = fmaf(u, kr[x], s[r][x]);
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < kRowsPerWarp; ++r) {
    const int row = warp + r * (kThreads / 32);
    if (row < dv) {
      float* p = Sn + (size_t)row * DK + lane * NPL;
      if (NPL == 4) {
        *reinterpret_cast<float4*>(p) = make_float4(s[r][0], s[r][1], s[r][2 % NPL], s[r][3 % NPL]);
      } else {
        *reinterpret_cast<float2*>(p) = make_float2(s[r][0], s[r][1]);
      }
    }
  }
}

// Programmatic dependent launch behind the verify kernel (which releases its dependents once the
// tree metadata it waited for is complete): the commit grid is scheduled as SMs drain, and every
// kernel launched this way orders itself with griddepcontrol.wait.  Behind any other kernel this
// is an ordinary launch.
cudaError_t launch_after_verify(void (*kernel)(const CommitArgs, const CommitLayers), int ctas, cudaStream_t stream,
                                const CommitArgs& a, const CommitLayers& tb, int threads = kRowThreads) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)ctas);
  cfg.blockDim = dim3((unsigned)threads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, a, tb);
}

}  // namespace

int tv_launch_commit(const CommitArgs& a, const CommitLayers& tb, cudaStream_t stream) {
  if (a.L < 1 || a.L > kCommitMaxLayers) return TV_ERR_BAD_ARG;
  const int items = a.L * a.B * a.H;
  if ((size_t)a.dk * a.dv > (size_t)kMaxVec * kThreads * 4) return TV_ERR_UNSUPPORTED;
  const bool recompute = a.rule == TV_GATED_DELTA && !a.has_U;
  static thread_local int sm_count = 0;
  if (!sm_count) {
    int dev = 0;
    TV_CUDA_TRY(cudaGetDevice(&dev));
    TV_CUDA_TRY(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev));
  }
  const int units = a.dv % kRowsPerCta == 0 ? items * (a.dv / kRowsPerCta) : 0;
  // the persistent kernel pays a prologue per CTA: worth it from about six units per CTA on
  if (!recompute && a.dk == 128 && units >= 6 * TV_STREAM_CTAS * sm_count && a.B <= kStreamMaxB &&
      a.tree.max_depth_all < kStreamMaxLen) {
    const int ctas = TV_STREAM_CTAS * sm_count;
    // ordinary launch: at this size the dependent launch measured slower (13.4 vs 12.7 ms per step
    // on 48 layers of 128 requests)
    if (a.bf16) commit_stream_dk128_kernel<true><<<ctas, kRowThreads, 0, stream>>>(a, tb);
    else commit_stream_dk128_kernel<false><<<ctas, kRowThreads, 0, stream>>>(a, tb);
  } else if (!recompute && a.dk == 128) {
    const int ctas = items * ((a.dv + kRowsPerCta - 1) / kRowsPerCta);
    TV_CUDA_TRY(a.bf16 ? launch_after_verify(commit_factored_dk128_kernel<true>, ctas, stream, a, tb)
                       : launch_after_verify(commit_factored_dk128_kernel<false>, ctas, stream, a, tb));
  } else if (!recompute) {
    TV_CUDA_TRY(a.bf16 ? launch_after_verify(commit_factored_kernel<true>, items, stream, a, tb, kThreads)
                       : launch_after_verify(commit_factored_kernel<false>, items, stream, a, tb, kThreads));
  } else if (a.dk == 128) {
    TV_CUDA_TRY(a.bf16 ? launch_after_verify(commit_delta_rows_kernel<true, 4>, items, stream, a, tb, kThreads)
                       : launch_after_verify(commit_delta_rows_kernel<false, 4>, items, stream, a, tb, kThreads));
  } else if (a.dk == 64) {
    TV_CUDA_TRY(a.bf16 ? launch_after_verify(commit_delta_rows_kernel<true, 2>, items, stream, a, tb, kThreads)
                       : launch_after_verify(commit_delta_rows_kernel<false, 2>, items, stream, a, tb, kThreads));
  } else {
    return TV_ERR_UNSUPPORTED;
  }
  TV_CUDA_TRY(cudaGetLastError());
  return TV_OK;
}
