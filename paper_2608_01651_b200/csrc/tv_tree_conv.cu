// Stage 1 of the per-layer pipeline (Section IV-C): tree-parallel causal depthwise convolution
// + bias + SiLU, optional q/k normalisation, gate preparation, and the head-major layout the
// verification kernels read -- one pass over the projected activations.
//
// Traffic is minimal (x is read once, q/k/v are written once), but per output element the
// operator needs W unpack+multiply-add pairs, a SiLU (two special-function operations) and its
// share of the row normalisation: about 20 instructions per 4 bytes moved, so on this GPU the
// kernel is bound by instruction issue before it is bound by HBM.  The design therefore spends
// its effort on instructions per element and on keeping the warps busy: persistent CTAs walk
// (request, head, q|k|v) slices so that the filter stays in registers; the rows of an item arrive
// as one TMA box one or two items ahead and are handed over through mbarriers, so the warps of a
// CTA never meet at a CTA-wide barrier; each half-warp derives the W tap rows of its own node rows
// from the parent array; and a half-warp owns a node row (8 channels per lane), so a row's sum of
// squares is a 4-step shuffle reduction and the row leaves as contiguous 16-byte stores.
#include <cuda_bf16.h>

#include "tv_internal.h"
#include "tv_tc_common.cuh"

namespace {

// Sixteen warps per SM (up to 128 registers, no spills: two CTAs of eight warps, four of four for
// trees of up to 64 nodes, eight of two up to 32) with the row loop unrolled twice measured faster
// than 24 warps at 80 registers.
constexpr int kConvUnroll = 2;
constexpr int kConvThreads = 256;
constexpr int kMaxConvDim = 256;

struct ConvArgs {
  const int32_t* parent;  // [n_trees][T]
  const int32_t* offsets; // packed forest: [B + 1] first row of each request (x rows and output planes); else null
  int32_t capacity;       // packed forest: rows of one output plane
  int32_t n_trees;
  int32_t B, H, T, dk, dv, W, normalize;
  int32_t slots;   // row buffers of a CTA (1..3): items requested slots - 1 ahead
  int32_t par_bulk; // the parents of a tree start on a 16-byte boundary and fill whole 16-byte units
  int32_t* status; // device status word of the tree (a wait that ran out is reported there)
  tvtc::FastDiv dB, dH;   // item -> (slice, request), slice -> (q|k|v, head)
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

// Lane geometry.  A node row of one 128-channel chunk is handled by 16 lanes with 8 channels
// each, as two groups of four.  bf16: the groups are adjacent (one 16-byte shared-memory read
// per tap and one 16-byte store).  f32: the groups sit 64 channels apart, so that each of the
// two 16-byte reads of a half-warp covers 256 contiguous bytes (no bank conflict).
template <typename IO> struct Geo;
template <> struct Geo<__nv_bfloat16> {
  static __device__ __forceinline__ int g0(int l16) { return 8 * l16; }
  static __device__ __forceinline__ int g1(int l16) { return 8 * l16 + 4; }
};
template <> struct Geo<float> {
  static __device__ __forceinline__ int g0(int l16) { return 4 * l16; }
  static __device__ __forceinline__ int g1(int l16) { return 64 + 4 * l16; }
};

__device__ __forceinline__ uint4 lds16(uint32_t addr) {
  uint4 r;
  asm("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
  return r;
}

// The eight staged values of this lane for one tap row; a0 / a1 are the shared-memory byte
// addresses of the lane's two channel groups in that row (bf16 reads both with one load).
__device__ __forceinline__ void load8(const __nv_bfloat16*, uint32_t a0, uint32_t, float (&o)[8]) {
  const uint4 t = lds16(a0);
  o[0] = __uint_as_float(t.x << 16); o[1] = __uint_as_float(t.x & 0xffff0000u);
  o[2] = __uint_as_float(t.y << 16); o[3] = __uint_as_float(t.y & 0xffff0000u);
  o[4] = __uint_as_float(t.z << 16); o[5] = __uint_as_float(t.z & 0xffff0000u);
  o[6] = __uint_as_float(t.w << 16); o[7] = __uint_as_float(t.w & 0xffff0000u);
}
__device__ __forceinline__ void load8(const float*, uint32_t a0, uint32_t a1, float (&o)[8]) {
  const uint4 a = lds16(a0), b = lds16(a1);
  o[0] = __uint_as_float(a.x); o[1] = __uint_as_float(a.y); o[2] = __uint_as_float(a.z); o[3] = __uint_as_float(a.w);
  o[4] = __uint_as_float(b.x); o[5] = __uint_as_float(b.y); o[6] = __uint_as_float(b.z); o[7] = __uint_as_float(b.w);
}
__device__ __forceinline__ void store8(__nv_bfloat16* row, int g0, int, bool live0, bool, const float (&y)[8]) {
  uint32_t p[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const __nv_bfloat162 t = __floats2bfloat162_rn(y[2 * e], y[2 * e + 1]);
    p[e] = *reinterpret_cast<const uint32_t*>(&t);
  }
  if (live0)
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(row + g0), "r"(p[0]), "r"(p[1]),
                 "r"(p[2]), "r"(p[3])
                 : "memory");
}
__device__ __forceinline__ void store8(float* row, int g0, int g1, bool live0, bool live1, const float (&y)[8]) {
  if (live0)
    asm volatile("st.global.L1::no_allocate.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(row + g0), "f"(y[0]), "f"(y[1]),
                 "f"(y[2]), "f"(y[3])
                 : "memory");
  if (live1)
    asm volatile("st.global.L1::no_allocate.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(row + g1), "f"(y[4]), "f"(y[5]),
                 "f"(y[6]), "f"(y[7])
                 : "memory");
}

// SiLU(z) = z / (1 + e^-z) in five instructions.  e^-z overflows to +inf for z < -88; its
// reciprocal is then 0 and the product -0.
__device__ __forceinline__ float silu(float z) {
  float e, r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(z * -1.4426950408889634f));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
  return z * r;
}
__device__ __forceinline__ float rsqrt_fast(float x) {
  float r;
  asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}

// Gate arithmetic on the special-function unit (ex2 / lg2 / rcp: relative error about 2^-22 each).
// softplus(z) = max(z, 0) + log(1 + e^-|z|): the rounding of 1 + e^-|z| leaves an absolute error of
// 6e-8, which the gate exp(-c * softplus) turns into a relative error of c * 6e-8.
__device__ __forceinline__ float exp_fast(float x) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x * 1.4426950408889634f));
  return r;
}
__device__ __forceinline__ float softplus(float z) {
  float l;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(l) : "f"(1.0f + exp_fast(-fabsf(z))));
  return fmaf(l, 0.6931471805599453f, fmaxf(z, 0.0f));
}
__device__ __forceinline__ float sigmoid_fast(float z) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + exp_fast(-z)));
  return r;
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}

// Work items are (slice, request) pairs, slice-major, where a slice is one head's q, k or v
// channels; a CTA walks a contiguous range of them, so its filter registers are reloaded only
// when the slice changes.  Shared memory:
//   NS x slot: [T][d] node rows (one TMA box of x) then [W-1][d] context rows, oldest first,
//   NS x [T] parents,
//   4 x ([128 NJ][W] filter taps + [128 NJ] bias) of a slice (3 x in the two-warp CTAs); every group of 8 channels is shifted
//   by two words, so that the 16 lanes of a row, which own 8 channels each, read 16 banks,
//   NS x (full, empty) mbarriers.
// The NW warps (eight, or four for trees of up to 64 nodes) run from item to item without a
// CTA-wide barrier.  Item n lives in slot n % NS.
// One warp (n % NW) requests item n + NS - 1 when it has finished item n (NS >= 3; with fewer slots,
// before it starts item n): the row box by TMA, the context rows and the parents by untiled bulk
// copies (unaligned parents and, when the slice changes, the filter by cp.async), all arriving on
// the slot's `full` barrier; before that it
// waits on the slot's `empty` barrier, on which every warp arrives when it has read the item that
// lived there.  Each half-warp derives the tap rows of the node rows it owns itself (lane k walks
// the parents of the half-warp's k-th row once per item; the row loop fetches them by shuffle),
// so nothing a warp needs is produced by another warp.
struct ConvItem {
  int slice, b, kind, h, d, c0;
  int n;          // node rows of this request
  int row0;       // first row of the request in x and in the gate inputs
  uint32_t orow;  // first row of this (request, head) in q/k/v and in the gate outputs
};

constexpr long long kConvDrainCycles = 1ll << 21;   // ~1 ms: copies still in flight after a timeout

template <typename IO, int W, int NJ, int NW>
__global__ void __launch_bounds__(NW * 32, (NJ == 1 && W <= 4) ? 16 / NW : 1)
tree_conv_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                 const ConvArgs a) {
  using namespace tvtc;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  constexpr int VEC = 16 / (int)sizeof(IO);
  const int T = a.T, H = a.H, B = a.B, dk = a.dk, dv = a.dv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, l16 = lane & 15, half = lane >> 4;
  const int C = H * (2 * dk + dv);
  const int dmax = dk > dv ? dk : dv;
  const int Tp = (T + 3) & ~3;
  const int NS = a.slots, PD = NS - 1;
  const bool issue_first = NS < 3;

  constexpr int kBiasAt = 128 * NJ * W + 32 * NJ;         // words
  constexpr int kFiltFloats = kBiasAt + 128 * NJ + 32 * NJ;
  const uint32_t slot_bytes = ((uint32_t)(T + W - 1) * dmax * sizeof(IO) + 127u) & ~127u;
  const uint32_t xs_u32 = smem_u32(smem_raw);
  const int32_t* par_s = reinterpret_cast<const int32_t*>(smem_raw + (size_t)NS * slot_bytes);   // [NS][Tp]
  // filter buffers: the items in flight (NS <= 3; two with two-warp CTAs) belong to NS slices at most
  constexpr int NF = NW == 2 ? 3 : 4;
  const float* filt_s = reinterpret_cast<const float*>(par_s + NS * Tp);                          // [NF][kFiltFloats]
  const uint32_t par_u32 = smem_u32(par_s), filt_u32 = smem_u32(filt_s);
  const uint32_t bar_u32 = filt_u32 + (uint32_t)NF * kFiltFloats * 4;   // full[NS], empty[NS] (8 bytes each)
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_raw + (bar_u32 - xs_u32) + 16 * NS);
  auto full_bar = [&](int s) { return bar_u32 + 8u * s; };
  auto empty_bar = [&](int s) { return bar_u32 + 8u * (NS + s); };

  if ((xs_u32 & 127u) != 0) {   // TMA wants its destination on a 128-byte boundary
    if (tid == 0 && a.status) atomicExch(a.status, (int)TV_ERR_CUDA);
    return;
  }
  const long long n_items = 3LL * H * B;
  const int first = (int)(n_items * blockIdx.x / gridDim.x);
  const int count = (int)(n_items * (blockIdx.x + 1) / gridDim.x) - first;
  if (count <= 0) return;
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(full_bar(s), 33);            // the issuing warp: expect_tx by lane 0, cp.async arrivals of 32 lanes
      mbar_init(empty_bar(s), NW);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Dependent launches on both sides: this kernel has come this far under the tail of the kernel
  // in front, whose output x may be; the kernel behind it may set itself up from here on (the
  // library's kernels read nothing this one writes before their own wait).  Dependents are
  // released after the wait, so that they never run beside anything older than this grid.
  __syncthreads();
  grid_dependency_wait();
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // An item's coordinates.  The cursor of the item being computed advances without divisions;
  // the warp that requests an item derives that item's coordinates from its number.
  auto set_slice = [&](ConvItem& it) {
    it.kind = (int)tvtc::fdiv((uint32_t)it.slice, a.dH);
    it.h = it.slice - it.kind * H;
    it.d = it.kind == 2 ? dv : dk;
    it.c0 = it.kind == 0 ? it.h * dk : it.kind == 1 ? (H + it.h) * dk : 2 * H * dk + it.h * dv;
  };
  // dense: request b owns rows b*T .. of x and the slab (b, h) of every output; packed forest:
  // rows offsets[b] .. of x and of every head's plane of `capacity` rows
  auto set_request = [&](ConvItem& it) {
    if (a.offsets == nullptr) {
      it.n = T;
      it.row0 = it.b * T;
      it.orow = (uint32_t)(it.b * H + it.h) * (uint32_t)T;
    } else {
      it.row0 = a.offsets[it.b];
      it.n = a.offsets[it.b + 1] - it.row0;
      it.orow = (uint32_t)it.h * (uint32_t)a.capacity + (uint32_t)it.row0;
    }
  };
  auto describe = [&](int item) {
    ConvItem it;
    it.slice = (int)tvtc::fdiv((uint32_t)item, a.dB);
    it.b = item - it.slice * B;
    set_slice(it);
    set_request(it);
    return it;
  };
  const int slice_first = (int)tvtc::fdiv((uint32_t)first, a.dB);
  ConvItem cur = describe(first);

  // The whole warp requests item m (descriptor `it`, slot m % NS).  False: a wait ran out.
  // `use` = m / NS, how often the slot has been filled before.
  auto issue = [&](int m, int slot, int use) -> bool {
    if (use > 0 && !mbar_wait_warp(empty_bar(slot), (uint32_t)((use - 1) & 1), abort_flag)) return false;
    const ConvItem it = describe(first + m);
    const int fc = it.slice - slice_first;   // slice changes since the CTA's first item: filter buffer fc % NF
    const bool new_filter = m == 0 || it.b == 0;
    const uint32_t dst = xs_u32 + (uint32_t)slot * slot_bytes;
    const uint32_t row_bytes = (uint32_t)it.d * sizeof(IO);
    // one thread: the row box (TMA), the W - 1 context rows and -- when its rows start on 16-byte
    // boundaries -- the parents as untiled bulk copies, all counted in bytes on the barrier
    const int32_t* psrc = a.parent + (size_t)(a.n_trees == 1 ? 0 : it.b) * T;
    const bool par_bulk = a.par_bulk != 0;
    if (lane == 0) {
      mbar_expect_tx(full_bar(slot), (uint32_t)(T + W - 1) * row_bytes + (par_bulk ? (uint32_t)T * 4u : 0u));
      tma_load_2d(dst, it.kind == 2 ? &map_v : &map_k, full_bar(slot), it.c0, it.row0);
      if (W > 1) {
        const IO* cb = reinterpret_cast<const IO*>(a.ctx) + (size_t)it.b * (W - 1) * C + it.c0;
#pragma unroll
        for (int r = 0; r < W - 1; ++r)
          bulk_load(dst + (uint32_t)(T + r) * row_bytes, cb + (size_t)r * C, row_bytes, full_bar(slot));
      }
      if (par_bulk) bulk_load(par_u32 + (uint32_t)(slot * Tp) * 4, psrc, (uint32_t)T * 4u, full_bar(slot));
    }
    if (!par_bulk)
      for (int i = lane; i < T; i += 32) cp_async4(par_u32 + (uint32_t)(slot * Tp + i) * 4, psrc + i);
    if (new_filter) {
      const uint32_t fdst = filt_u32 + (uint32_t)((fc % NF) * kFiltFloats) * 4;
      const float* wsrc = a.weight + (size_t)it.c0 * W;
      for (int c = lane; c < it.d; c += 32) {
        const uint32_t shift = 2 * (c >> 3);
#pragma unroll
        for (int t = 0; t < W; ++t) cp_async4(fdst + (c * W + t + shift) * 4, wsrc + c * W + t);
        if (a.bias != nullptr) cp_async4(fdst + (kBiasAt + c + shift) * 4, a.bias + it.c0 + c);
      }
    }
    cp_async_arrive(full_bar(slot));
    return true;
  };

  // ---- prologue: the first PD items (the first one when there is a single slot)
  {
    const int ahead = PD > 0 ? PD : 0;
    for (int m = 0; m < ahead && m < count; ++m)
      if (warp == (m & (NW - 1))) issue(m, m, 0);
  }

  // this thread's gate input of an item (alpha with the q slice, beta with the k slice), loaded
  // one item ahead
  auto fetch_gate = [&](const ConvItem& it) -> IO {
    const void* src = it.kind == 0 ? a.gate_a : it.kind == 1 ? a.gate_b : nullptr;
    if (src == nullptr || tid >= it.n) return IO(0.0f);
    return reinterpret_cast<const IO*>(src)[(uint32_t)(it.row0 + tid) * (uint32_t)H + (uint32_t)it.h];
  };
  IO gate_next = fetch_gate(cur);

  // Dead channel groups (past the slice's width) keep zero weights and read the row's first
  // bytes, so the row loop is straight-line code; only their store is predicated off.
  float wreg[NJ][W][8], breg[NJ][8];
  bool live0[NJ], live1[NJ];
  uint32_t off0[NJ], off1[NJ];
  int loaded_slice = -1;
  const float eps = a.eps;
  const bool want_norm = a.normalize != 0;
  bool ok = true;
  int slot = 0, n = 0;
  int pre_slot = PD, pre_use = 0;   // slot of item n + PD and how often it has been filled
  uint32_t phase = 0;               // parity of the slot's `full` barrier for item n

  for (; n < count; ++n) {
    if (issue_first && n + PD < count) {
      if (warp == ((n + PD) & (NW - 1)) && !issue(n + PD, pre_slot, pre_use)) { ok = false; break; }
    }
    if (!mbar_wait_warp(full_bar(slot), phase, abort_flag)) { ok = false; break; }
    const int d = cur.d;
    const uint32_t row_bytes = (uint32_t)d * sizeof(IO);

    // ---- this lane's filter taps and bias, when the slice changes
    if (cur.slice != loaded_slice) {
      loaded_slice = cur.slice;
      const float* wf = filt_s + ((cur.slice - slice_first) % NF) * kFiltFloats;
      const float* bf = wf + kBiasAt;
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        const int g0 = 128 * j + Geo<IO>::g0(l16), g1 = 128 * j + Geo<IO>::g1(l16);
        live0[j] = g0 < d;
        live1[j] = g1 < d;
        off0[j] = live0[j] ? (uint32_t)(g0 * sizeof(IO)) : 0u;
        off1[j] = live1[j] ? (uint32_t)(g1 * sizeof(IO)) : 0u;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int c = e < 4 ? g0 + e : g1 + e - 4;
          const bool live = e < 4 ? live0[j] : live1[j];
          const int shift = 2 * (c >> 3);
          breg[j][e] = live && a.bias ? bf[c + shift] : 0.0f;
#pragma unroll
          for (int r = 0; r < W; ++r) wreg[j][r][e] = live ? wf[c * W + (W - 1 - r) + shift] : 0.0f;
        }
      }
    }

    // ---- gate preparation for this (request, head): alpha with the q slice, beta with the k
    // slice (the work is spread over the CTAs of two thirds of the slices); the input was
    // requested one item ago.
    const bool do_alpha = cur.kind == 0 && a.gate_a != nullptr && tid < cur.n;
    const bool do_beta = cur.kind == 1 && a.gate_b != nullptr && tid < cur.n;
    const IO gate_raw = gate_next;
    float gate_A = 0.f, gate_dt = 0.f;
    if (do_alpha) {
      gate_A = __ldg(a.A_log + cur.h);
      gate_dt = __ldg(a.dt_bias + cur.h);
    }

    // ---- tap rows: lane k of a half-warp walks the parents of the half-warp's k-th row
    const int Tn = cur.n;
    const uint32_t xs_item = xs_u32 + (uint32_t)slot * slot_bytes;
    uint32_t mytap[W];
    {
      const int32_t* par = par_s + slot * Tp;
      int j = 2 * warp + half + 2 * NW * l16, ctx_row = W - 2;
      if (j >= Tn) j = Tn - 1;   // rows past the end repeat the last one (computed, not stored)
#pragma unroll
      for (int r = 0; r < W; ++r) {
        int row;
        if (j >= 0) {
          row = j;
          j = par[j];
        } else {
          row = T + ctx_row--;
        }
        mytap[r] = (uint32_t)row * row_bytes;
      }
    }

    // ---- each half-warp takes one node row at a time
    IO* out = reinterpret_cast<IO*>(cur.kind == 0 ? a.q : cur.kind == 1 ? a.k : a.v) + (size_t)cur.orow * d;
    const bool norm = want_norm && cur.kind < 2;
    uint32_t base0[NJ], base1[NJ];
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
      base0[j] = xs_item + off0[j];
      base1[j] = xs_item + off1[j];
    }
    int src_lane = lane & 16;
#pragma unroll kConvUnroll
    for (int i0 = 2 * warp; i0 < Tn; i0 += 2 * NW, ++src_lane) {
      const bool row_live = i0 + half < Tn;
      const int i = row_live ? i0 + half : Tn - 1;
      uint32_t tap[W];
#pragma unroll
      for (int r = 0; r < W; ++r) tap[r] = __shfl_sync(0xffffffffu, mytap[r], src_lane);
      float y[NJ][8];
      float ss = 0.0f;
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
#pragma unroll
        for (int r = 0; r < W; ++r) {
          float in[8];
          load8((const IO*)nullptr, base0[j] + tap[r], base1[j] + tap[r], in);
#pragma unroll
          for (int e = 0; e < 8; ++e) y[j][e] = fmaf(wreg[j][r][e], in[e], r == 0 ? breg[j][e] : y[j][e]);
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          y[j][e] = silu(y[j][e]);
          ss = fmaf(y[j][e], y[j][e], ss);
        }
      }
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      const float sc = norm ? rsqrt_fast(ss + eps) : 1.0f;
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
#pragma unroll
        for (int e = 0; e < 8; ++e) y[j][e] *= sc;
        store8(out + (uint32_t)(i * d + 128 * j), Geo<IO>::g0(l16), Geo<IO>::g1(l16), row_live && live0[j],
               row_live && live1[j], y[j]);
      }
    }
    // this warp has read the slot
    __syncwarp();
    if (lane == 0) mbar_arrive(empty_bar(slot));

    if (do_alpha) a.alpha[cur.orow + tid] = exp_fast(-exp_fast(gate_A) * softplus(to_f32(gate_raw) + gate_dt));
    if (do_beta) a.beta[cur.orow + tid] = sigmoid_fast(to_f32(gate_raw));

    if (!issue_first && n + PD < count) {
      if (warp == ((n + PD) & (NW - 1)) && !issue(n + PD, pre_slot, pre_use)) { ok = false; break; }
    }
    if (++pre_slot == NS) {
      pre_slot = 0;
      ++pre_use;
    }
    if (n + 1 < count) {
      if (++cur.b == B) {
        cur.b = 0;
        ++cur.slice;
        set_slice(cur);
      }
      set_request(cur);
      gate_next = fetch_gate(cur);
    }
    if (++slot == NS) {
      slot = 0;
      phase ^= 1;
    }
  }

  if (!ok) {
    // A wait ran out (or another warp's did).  Copies requested for the items this warp has not
    // consumed may still be in flight: give them a moment before the CTA's memory is released.
    int dummy = 0;
    for (int m = n; m <= n + PD && m < count; ++m)
      mbar_wait(full_bar(m % NS), (uint32_t)((m / NS) & 1), &dummy, kConvDrainCycles);
    asm volatile("cp.async.wait_all;" ::: "memory");
    if (lane == 0 && a.status) atomicExch(a.status, (int)TV_ERR_DEVICE_TIMEOUT);
  }
}

// Context rows after the commit: one thread per 16-byte channel vector reads its W-1 source
// values (accepted node and its ancestors first, then the old context) before it writes any, so
// ctx_new may be ctx itself.
template <typename IO, int W>
__global__ void __launch_bounds__(kConvThreads)
conv_commit_kernel(const int32_t* __restrict__ parent, int32_t n_trees, const int32_t* __restrict__ offsets,
                   const int32_t* __restrict__ accepted, int32_t T, int32_t C, const IO* x, const IO* ctx,
                   IO* ctx_new) {
  constexpr int VEC = 16 / (int)sizeof(IO);
  tvtc::grid_dependency_wait();   // dependent launch: nothing is read before the kernel in front is done
  const int b = blockIdx.y;
  const int col = (blockIdx.x * kConvThreads + threadIdx.x) * VEC;
  if (col >= C) return;
  int acc = accepted[b];
  const int row0 = offsets ? offsets[b] : b * T;                     // packed forest: the request's first x row
  const int nb = offsets ? offsets[b + 1] - offsets[b] : T;
  if (acc >= nb) acc = -1;
  const int32_t* par = parent + (size_t)(n_trees == 1 ? 0 : b) * T;
  const IO* xb = x + (size_t)row0 * C + col;
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
  if (d->impl != TV_IMPL_AUTO && d->impl != TV_IMPL_SIMT && d->impl != TV_IMPL_TC) return TV_ERR_BAD_ARG;
  if (d->impl == TV_IMPL_TC) return TV_ERR_UNSUPPORTED;   // no tensor-core form of this operator
  if (d->T > TV_MAX_NODES || d->dk > kMaxConvDim || d->dv > kMaxConvDim || d->W > TV_CONV_MAX_TAPS)
    return TV_ERR_UNSUPPORTED;
  const int m = d->io_dtype == TV_BF16 ? 7 : 3;
  if ((d->dk & m) || (d->dv & m)) return TV_ERR_UNSUPPORTED;
  if (t->n != d->T) return TV_ERR_BAD_ARG;
  if (t->n_trees != 1 && t->n_trees != d->B) return TV_ERR_BAD_ARG;
  if (!t->offsets.empty() && t->n_trees != d->B) return TV_ERR_BAD_ARG;
  if ((int64_t)d->B * d->H * 3 > 0x7fffffffLL || d->B > 65535) return TV_ERR_UNSUPPORTED;
  // rows of an output plane and gate elements are indexed in 32 bits
  const int64_t out_rows = t->offsets.empty() ? (int64_t)d->B * d->H * d->T : (int64_t)d->H * t->capacity;
  if (out_rows > 0x7fffffffLL) return TV_ERR_UNSUPPORTED;
  if (!t->uploaded) return TV_ERR_NOT_UPLOADED;
  return TV_OK;
}

template <typename IO, int W>
int launch_conv(const ConvArgs& a_in, cudaStream_t stream) {
  ConvArgs a = a_in;
  constexpr bool kTwoPerSm = W <= 4;   // and d <= 128: the kernel's launch bounds
  const int dmax = a.dk > a.dv ? a.dk : a.dv;
  const int NJ = dmax <= 128 ? 1 : 2;
  const size_t slot = ((size_t)(a.T + W - 1) * dmax * sizeof(IO) + 127) & ~(size_t)127;
  auto smem_for = [&](int ns) {
    return ns * slot + (size_t)ns * ((a.T + 3) & ~3) * 4 + 4 * (size_t)NJ * (128 * (W + 1) + 64) * 4 + 16 * ns + 16;
  };
  // three slots with two CTAs per SM if that fits (a fourth measured slower: 41.4 against 39.4 us
  // on B = 32, T = 64), else as many slots, up to three, as fit a CTA that has the SM's shared
  // memory to itself
  const size_t half_sm = 112 * 1024, whole_sm = 226 * 1024;
  if (kTwoPerSm && NJ == 1 && smem_for(3) <= half_sm) a.slots = 3;
  else a.slots = smem_for(3) <= whole_sm ? 3 : smem_for(2) <= whole_sm ? 2 : 1;
  // Up to 64 nodes: CTAs of four warps, four per SM, two slots each.  A warp then takes twice as
  // many rows of an item, which halves the per-item part of its work (a third of an item at 64
  // nodes with eight warps): 39.4 -> 37.4 us on B = 32, T = 64 and 84.3 -> 66.1 us on B = 128,
  // T = 32.  At 128 nodes the four CTAs' slots do not fit.
  const bool small = kTwoPerSm && NJ == 1 && a.T <= 64 && smem_for(2) <= 55 * 1024;
  // up to 32 nodes: CTAs of two warps, eight per SM, by the same argument
  // (three filter buffers instead of four there: one fewer than smem_for() counts)
  const size_t filt_bytes = (size_t)(128 * (W + 1) + 64) * 4;
  const bool tiny = small && a.T <= 32 && smem_for(2) - filt_bytes <= 27 * 1024;
  if (small) a.slots = 2;
  const size_t smem = smem_for(a.slots) - (tiny ? filt_bytes : 0);
  if (smem > whole_sm) return TV_ERR_UNSUPPORTED;
  // x as a [rows][C] tensor; one box = the T node rows of a request x the d channels of a slice
  const int C = a.H * (2 * a.dk + a.dv);
  const uint64_t rows = a.offsets ? (uint64_t)a.capacity : (uint64_t)a.B * a.T;
  const CUtensorMapDataType dt = sizeof(IO) == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  // A serving loop calls with the same buffers and shapes round after round: the two tensor maps
  // and what the runtime says about the kernel (SM count, CTAs per SM at this shared-memory size)
  // are kept per thread for the last call's arguments.
  struct MapCache {
    const void* x = nullptr;
    uint64_t rows = 0;
    int C = 0, dk = 0, dv = 0, T = 0;
    alignas(64) CUtensorMap map_k, map_v;
  };
  struct LaunchCache {
    const void* kernel = nullptr;
    size_t smem = 0;
    int dev = -1, sms = 0, per_sm = 0;
  };
  static thread_local MapCache mc;
  static thread_local LaunchCache lc;
  if (mc.x != a.x || mc.rows != rows || mc.C != C || mc.dk != a.dk || mc.dv != a.dv || mc.T != a.T) {
    mc.x = nullptr;
    if (!tvtc::make_map2_plain(&mc.map_k, a.x, dt, sizeof(IO), rows, C, a.dk, a.T) ||
        !tvtc::make_map2_plain(&mc.map_v, a.x, dt, sizeof(IO), rows, C, a.dv, a.T))
      return TV_ERR_CUDA;
    mc.x = a.x; mc.rows = rows; mc.C = C; mc.dk = a.dk; mc.dv = a.dv; mc.T = a.T;
  }
  const CUtensorMap &map_k = mc.map_k, &map_v = mc.map_v;
  int dev = 0;
  TV_CUDA_TRY(cudaGetDevice(&dev));
  auto go = [&](auto kernel, int threads) -> int {
    if (lc.kernel != (const void*)kernel || lc.smem != smem || lc.dev != dev) {
      lc.kernel = nullptr;
      TV_CUDA_TRY(cudaDeviceGetAttribute(&lc.sms, cudaDevAttrMultiProcessorCount, dev));
      if (smem > 48 * 1024)
        TV_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      TV_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&lc.per_sm, kernel, threads, smem));
      lc.kernel = (const void*)kernel; lc.smem = smem; lc.dev = dev;
    }
    const int sms = lc.sms, per_sm = lc.per_sm;
    if (per_sm < 1) return TV_ERR_UNSUPPORTED;
    const long long items = 3LL * a.H * a.B, slots = (long long)sms * per_sm;
    const unsigned grid = (unsigned)(items < slots ? items : slots);
    TV_CUDA_TRY(tvtc::launch_dependent(kernel, (int)grid, threads, smem, stream, map_k, map_v, a));
    return TV_OK;
  };
  if (tiny) return go(tree_conv_kernel<IO, W, 1, 2>, 64);
  if (small) return go(tree_conv_kernel<IO, W, 1, 4>, 128);
  return NJ == 1 ? go(tree_conv_kernel<IO, W, 1, 8>, 256) : go(tree_conv_kernel<IO, W, 2, 8>, 256);
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
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kConvThreads);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  TV_CUDA_TRY(cudaLaunchKernelEx(&cfg, conv_commit_kernel<IO, W>, (const int32_t*)t->d_parent, (int32_t)t->n_trees,
                                 (const int32_t*)t->d_offsets, accepted, (int32_t)d->T, (int32_t)C, (const IO*)x,
                                 (const IO*)ctx, (IO*)ctx_new));
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
      !aligned16(weight) || !aligned16(bias) || ((uintptr_t)alpha & 3) || ((uintptr_t)beta & 3) ||
      ((uintptr_t)A_log & 3) || ((uintptr_t)dt_bias & 3))
    return TV_ERR_BAD_ARG;
  const uintptr_t esz = d->io_dtype == TV_BF16 ? 2 : 4;
  if (((uintptr_t)gate_a & (esz - 1)) || ((uintptr_t)gate_b & (esz - 1))) return TV_ERR_BAD_ARG;
  if (q == x || k == x || v == x || q == k || q == v || k == v) return TV_ERR_BAD_ARG;
  ConvArgs a;
  a.parent = tree->d_parent; a.n_trees = tree->n_trees;
  a.offsets = tree->d_offsets; a.capacity = tree->capacity;
  a.B = d->B; a.H = d->H; a.T = d->T; a.dk = d->dk; a.dv = d->dv; a.W = d->W;
  a.normalize = d->normalize_qk != 0; a.eps = d->eps; a.slots = 0; a.status = tree->d_status;
  a.par_bulk = (d->T % 4 == 0) && aligned16(tree->d_parent);
  a.dB = tvtc::make_fastdiv((uint32_t)d->B); a.dH = tvtc::make_fastdiv((uint32_t)d->H);
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
