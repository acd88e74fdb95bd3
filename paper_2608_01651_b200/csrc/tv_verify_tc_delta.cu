// Tree verification of the gated delta rule on the tensor cores (tcgen05 + TMEM + TMA).
//
// Shapes: bf16 q/k/v, fp32 state, dk = dv = 128, T <= 64, tree depth <= 15.
//
// Theorem 1 (Eq. 2) regrouped so that the state is contracted once (a WY-style
// factorisation restricted to ancestor sets).  With N = (I+G)^-1 (Lemma 2/3),
// A = N D_beta, W = C A:
//     O = Q_eff S_pre^T + W V,   Q_eff = D_P Q - (W D_P) K
//     U = A V - K_eff S_pre^T,   K_eff = (A D_P) K
// G, C, N, A, W are T x T but ancestor-sparse: row i has entries only on the
// root-to-node path p_0 < ... < p_d = i of node i, and slot s of node i and of
// any descendant refer to the same node p_s.  Row i of W = C N D_beta and of
// A = N D_beta come from ONE back-substitution each on the path-restricted unit
// lower-triangular system (w L = c, x L = e_d; L = I + G on the path): d^2/2
// FMAs per row, no T x T product, no Neumann rounds, no level barriers.  All
// decay factors are products of alpha over a stretch of the row's own path
// (P_t / P_s for ancestors s < t, never a quotient of two underflowing
// numbers), built up one factor at a time beside the back-substitution.
//
// Tile rows 0..63 carry the O problem of node i, rows 64..127 the U problem of
// node i (the M = 128 MMA shape is otherwise half empty at T <= 64).  Q and K
// are stacked in one operand tile [Q ; K]:
//     Sc  = [Q ; K] K^T   (bf16, N = 64)   rows 0..63 = Q K^T, rows 64..127 = K K^T
//     E1: path-sparse raw rows of C and G; E2: back-substitution, operand tiles
//     Qf  = D_P Q   (rows 0..63; written to TMEM by the threads that know P_i, in fp32)
//         + [-(W D_P) ; -(A D_P)] K        rows 0..63 = Q_eff, rows 64..127 = -K_eff
//           (bf16 hi/lo coefficients, accumulated into the same TMEM columns)
//     acc = Qf S_pre^T (tf32, A operand straight from TMEM) + [W ; A] V (bf16 hi/lo)
//     O = acc[0..63], U = acc[64..127]
// The [Q ; K] tile is double-buffered and its Gram product is issued one item ahead, so the load
// and the product of item n+1 run under the row solve of item n; what bounds an item is then the
// CUDA-core chain of the eight compute warps: E1 -> path gather -> output staging of the previous
// item -> back-substitution -> Qf initialisation -> operand tiles.  Loads, MMA issue, output
// stores and the per-item tables (masks, gates) each have a warp of their own.
// S_pre goes TMA -> shared memory -> tensor core untouched; O and U leave
// through swizzled staging chunks and TMA stores.  Every wait is a bounded
// mbarrier wait (status word on expiry); every TMA load is a plain per-CTA copy.
#include "tv_tc_common.cuh"

namespace {

using namespace tvtc;

constexpr int kThreads = 384;     // producer, MMA issuer, 8 compute warps, output-store warp, metadata warp
constexpr int kComputeWarps = 8;
constexpr int kSlots = 16;     // path slots per node: depth <= 15
constexpr int kRows = 64;      // T <= 64
constexpr int kLd = 17;        // row stride of the slot tables (floats): conflict-free per slot
constexpr int kLdP = 20;       // row stride of the path table (bytes)

// shared memory map (bytes from the 1024-aligned base); 14 tiles of 128 rows x 128 B
constexpr uint32_t kOffQK = 0;                   // buffer 0 of [Q ; K]: 2 k-halves, rows 0..63 Q, rows 64..127 K
constexpr uint32_t kOffV = 2 * kTile;            // 2 dv-halves of V (rows 0..63); upper halves: scratch
constexpr uint32_t kOffS = 4 * kTile;            // 4 k-chunks of S_pre [128 v][32] f32
constexpr uint32_t kOffQK1 = 8 * kTile;          // buffer 1 of [Q ; K] (items alternate between the two)
constexpr uint32_t kOffAk = 10 * kTile;          // hi, lo of [-(W D_P) ; -(A D_P)]  [128][64] bf16
constexpr uint32_t kOffW = 12 * kTile;           // hi, lo of [W ; A]                [128][64] bf16
constexpr uint32_t kOffStage = kOffAk;           // 8 output chunks of 8 KiB (O: 0..3, U: 4..7)
constexpr uint32_t kOffGs = kOffV + 8192;        // float Gs[64][kLd]: raw K K^T on the path
constexpr uint32_t kOffCs = kOffV + kTile + 8192;  // float Cs[64][kLd]: raw Q K^T on the path
constexpr uint32_t kOffSmall = kOffCs + 4352;    // 2 buffers x {float al[64] (alpha), be[64] (beta)}
constexpr uint32_t kOffMeta = kOffGs + 4352;     // 2 buffers x uint64 strict-ancestor mask [64]
constexpr uint32_t kOffPs = kOffMeta + 1024;     // 2 buffers x uint8 Ps[64][kLdP]: path nodes in slot order
constexpr uint32_t kOffBar = 14 * kTile;
constexpr uint32_t kOffMisc = kOffBar + 8 * 24;
constexpr uint32_t kSmemBytes = kOffMisc + 64 + 1024;

enum Bar {
  QK_FULL = 0, QK_FREE, S_FULL, S_FREE, V_FULL, V_FREE,
  G_DONE, G_FREE, W_READY, D1_DONE, ACC_DONE, ACC_FREE, E1_SYNC,
  OST_READY, OST_FREE, QK_FULL1, QK_FREE1, META_FULL, META_FULL1, META_FREE, META_FREE1
};

constexpr uint32_t kColSc = 0, kColQf = 128, kColAcc = 256;
// The tensor core cuts a tf32 operand to 10 explicit mantissa bits by dropping the rest (towards
// zero).  A value whose mantissa is spread evenly loses 2^-11 ln 2 of its magnitude on average,
// so the state product Qf S_pre^T, both of whose operands are cut, comes out 2 * 2^-11 ln 2 =
// 6.8e-4 short on average: a bias, the same sign everywhere, and the largest part of this kernel's
// error (measured: O 9e-4 -> 4e-4 on fresh states, S_new 4.7e-4 -> 4e-5 after thousands of
// commits once it is taken out; the optimum found by scanning the constant is the predicted one).
// Qf is scaled up by that factor where it is produced (the D_P Q rows and the coefficient tile of
// the key product), which leaves the zero-mean part of the rounding.
constexpr float kTf32Comp = 1.0f + 6.7697e-4f;

struct DeltaParams {
  TreeDev tree;
  int32_t n_items, B, H, T;
  int32_t Hk;  // q/k heads (grouped key heads); H when not grouped
  const float* alpha;
  const float* beta;
  int32_t want_U;
  int32_t* status;
  // packed forest only (see tv_verify_tc.cu): row offsets of the requests, rows per plane, and the
  // outputs as plain pointers for the rows that leave from registers
  const int32_t* offsets;
  int32_t capacity;
  ItemDiv div;   // divisions by H, B, H / Hk as multiply-shift
  Str3 gate;     // strides of alpha and beta (dense layouts)
  // The q, k, v, O, U maps are 4-D, (channel, node, head, layer*request) or (channel, head, node, ...)
  // whichever has ascending strides: bit 0 / 1 / 2 set = q,k / v / O,U take the node coordinate first.
  int32_t node_first;
  float* O;
  float* U;
};

// bf16 hi/lo parts of x (hi = upper 16 bits, lo = upper 16 bits of the exact remainder)
__device__ __forceinline__ void split_bf16(float x, uint16_t& hi, uint16_t& lo) {
  const uint32_t b = __float_as_uint(x);
  const uint32_t h = b & 0xffff0000u;
  hi = (uint16_t)(h >> 16);
  lo = (uint16_t)(__float_as_uint(x - __uint_as_float(h)) >> 16);
}

// DMAX: compile-time bound on the tree depth (8 covers draft trees, 15 the rest), so that the
// per-row triangular solve is straight-line code whose loads all issue up front.
// PACKED = packed forest: loads take the 64-row box at the request's offset, stores are cut to
// the request's node count (TMA boxes of 64/32/16/8 rows, then a register tail), and operand
// rows past the last node of the forest are zeroed in shared memory before they meet a zero
// coefficient.  The dense instantiation is given the 64-row maps for all box sizes and ignores them.
struct OutMaps {
  CUtensorMap m64, m32, m16, m8;
};
template <int DMAX, bool PACKED>
__global__ void __launch_bounds__(kThreads, 1)
verify_tc_delta_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmS,
                       const __grid_constant__ OutMaps mapsO, const __grid_constant__ OutMaps mapsU,
                       const DeltaParams p) {
  const CUtensorMap& tmO = mapsO.m64;
  const CUtensorMap& tmU = mapsU.m64;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(sm);
  float* Gs = reinterpret_cast<float*>(sm + kOffGs);
  float* Cs = reinterpret_cast<float*>(sm + kOffCs);
  uint8_t* Ps_all = reinterpret_cast<uint8_t*>(sm + kOffPs);     // [2][64][kLdP]
  float* tab_s = reinterpret_cast<float*>(sm + kOffSmall);       // [2][la[64], be[64]]
  uint64_t* mask_s = reinterpret_cast<uint64_t*>(sm + kOffMeta);   // [2][64]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + kOffMisc + 4);
  auto bar = [&](int i) { return sbase + kOffBar + 8u * i; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int T = p.T;
  const bool want_U = p.want_U != 0;
  const bool nf_qk = p.node_first & 1, nf_v = p.node_first & 2, nf_o = p.node_first & 4;
  // box coordinates of an item: q/k head, v/O/U head, outermost index (layer*request, or the layer
  // of a packed forest) and the first node row
  struct Coord {
    int hq, h, z, y0;
  };
  auto coord_of = [&](int item) -> Coord {
    Coord c;
    const int lb = (int)fdiv((uint32_t)item, p.div.dH);
    c.h = item - lb * p.H;
    c.hq = (int)fdiv((uint32_t)c.h, p.div.dG);
    c.z = lb;
    c.y0 = 0;
    if constexpr (PACKED) {
      const int l = (int)fdiv((uint32_t)lb, p.div.dB);
      c.z = l;
      c.y0 = p.offsets[lb - l * p.B];
    }
    return c;
  };

  if (tid == 0) {
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    mbar_init(bar(QK_FULL), 1);  mbar_init(bar(QK_FREE), 1);
    mbar_init(bar(QK_FULL1), 1); mbar_init(bar(QK_FREE1), 1);
    mbar_init(bar(S_FULL), 1);   mbar_init(bar(S_FREE), 1);
    mbar_init(bar(V_FULL), 1);   mbar_init(bar(V_FREE), 1);
    mbar_init(bar(G_DONE), 1);   mbar_init(bar(G_FREE), kComputeWarps);
    mbar_init(bar(W_READY), kComputeWarps);
    mbar_init(bar(D1_DONE), 1);
    mbar_init(bar(ACC_DONE), 1); mbar_init(bar(ACC_FREE), kComputeWarps);
    mbar_init(bar(META_FULL), 1);  mbar_init(bar(META_FULL1), 1);
    mbar_init(bar(META_FREE), kComputeWarps); mbar_init(bar(META_FREE1), kComputeWarps);
    mbar_init(bar(E1_SYNC), kComputeWarps);
    mbar_init(bar(OST_READY), kComputeWarps);
    mbar_init(bar(OST_FREE), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      // ===================== TMA producer =====================
      int pend_qk = 0, pend_qk_bar = QK_FULL, pend_s = 0, pend_v = 0;
      uint32_t it = 0;
      grid_dependency_wait();   // inputs may come from the kernel in front (dependent launch)
      for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++it) {
        const uint32_t ph = it & 1;
        // [Q ; K] is double-buffered: item it uses buffer it & 1, each buffer's barriers flip
        // every second item
        const int qb = (int)(it & 1);
        const uint32_t qph = (it >> 1) & 1;
        const uint32_t qk_base = qb ? kOffQK1 : kOffQK;
        const int qfull = qb ? QK_FULL1 : QK_FULL, qfree = qb ? QK_FREE1 : QK_FREE;
        if (!mbar_wait(bar(qfree), qph ^ 1, abort_flag)) break;
        mbar_expect_tx(bar(qfull), 4 * 8192);
        const Coord co = coord_of(item);
        load_box(sbase + qk_base, &tmQ, bar(qfull), nf_qk, 0, co.y0, co.hq, co.z);
        load_box(sbase + qk_base + kTile, &tmQ, bar(qfull), nf_qk, 64, co.y0, co.hq, co.z);
        load_box(sbase + qk_base + 8192, &tmK, bar(qfull), nf_qk, 0, co.y0, co.hq, co.z);
        load_box(sbase + qk_base + kTile + 8192, &tmK, bar(qfull), nf_qk, 64, co.y0, co.hq, co.z);
        pend_qk_bar = qfull;
        pend_qk = 1 + (int)qph;
        if (!mbar_wait(bar(S_FREE), ph ^ 1, abort_flag)) break;
        mbar_expect_tx(bar(S_FULL), 4 * kTile);
#pragma unroll
        for (int c = 0; c < 4; ++c)
          tma_load_3d(sbase + kOffS + c * kTile, &tmS, bar(S_FULL), 32 * c, 0, item);
        pend_s = 1 + (int)ph;
        if (!mbar_wait(bar(V_FREE), ph ^ 1, abort_flag)) break;
        mbar_expect_tx(bar(V_FULL), 2 * 8192);
        load_box(sbase + kOffV, &tmV, bar(V_FULL), nf_v, 0, co.y0, co.h, co.z);
        load_box(sbase + kOffV + kTile, &tmV, bar(V_FULL), nf_v, 64, co.y0, co.h, co.z);
        pend_v = 1 + (int)ph;
      }
      if (*abort_flag) {
        if (pend_qk) mbar_wait(bar(pend_qk_bar), pend_qk - 1, abort_flag + 1);
        if (pend_s) mbar_wait(bar(S_FULL), pend_s - 1, abort_flag + 1);
        if (pend_v) mbar_wait(bar(V_FULL), pend_v - 1, abort_flag + 1);
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    if (lane == 0) {
      constexpr uint32_t kIdGram = idesc_bf16(64, false);
      constexpr uint32_t kIdMn = idesc_bf16(128, true);
      constexpr uint32_t kIdTf32 = idesc_tf32(128);
      // Sc = [Q ; K] K^T of local item j, issued one item ahead of the rest of the chain so that
      // it runs under the row solve of the item before
      const uint32_t n_local = p.n_items > (int)blockIdx.x
                                   ? (uint32_t)((p.n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x) : 0u;
      auto gram = [&](uint32_t j) -> bool {
        const uint32_t qk_base = (j & 1) ? kOffQK1 : kOffQK;
        if (!mbar_wait(bar((j & 1) ? QK_FULL1 : QK_FULL), (j >> 1) & 1, abort_flag)) return false;
        if (!mbar_wait(bar(G_FREE), (j & 1) ^ 1, abort_flag)) return false;   // score columns read by E1 of j-1
        tc_fence_after();
        // (the MMA loops are kept rolled, descriptor = base + step: the roles of a CTA share one
        // instruction cache)
        const uint64_t dA = desc_kmajor(sbase + qk_base), dB = desc_kmajor(sbase + qk_base + 8192);
#pragma unroll
        for (uint32_t i = 0; i < 8; ++i) {   // k half i >> 2, 32 bytes of k per step
          const uint32_t off = ((i >> 2) * kTile + (i & 3u) * 32u) >> 4;
          mma_bf16_ss(tmem + kColSc, dA + off, dB + off, kIdGram, i);
        }
        tc_commit(bar(G_DONE));
        return true;
      };
      bool mma_ok = n_local == 0 || gram(0);
      for (uint32_t it = 0; mma_ok && it < n_local; ++it) {
        const uint32_t ph = it & 1;
        const uint32_t qk_base = (it & 1) ? kOffQK1 : kOffQK;
        if (it + 1 < n_local && !gram(it + 1)) break;
        // Qf += -(W D_P) K  (rows 64..127: -(A D_P) K); the compute warps initialised Qf with D_P Q
        if (!mbar_wait(bar(W_READY), ph, abort_flag)) break;
        tc_fence_after();
        {
          const uint64_t dAk = desc_kmajor(sbase + kOffAk), dKr = desc_mnmajor(sbase + qk_base + 4 * 2048, kTile);
#pragma unroll
          for (uint32_t i = 0; i < 8; ++i)   // part i >> 2 (hi, lo), K rows 16 (i & 3) .. of the stacked tile
            mma_bf16_ss(tmem + kColQf, dAk + (((i >> 2) * kTile + (i & 3u) * 32u) >> 4),
                        dKr + (((i & 3u) * 2048u) >> 4), kIdMn, 1);
        }
        tc_commit(bar(D1_DONE));
        tc_commit(bar((it & 1) ? QK_FREE1 : QK_FREE));
        // acc = Qf S_pre^T: Qf must be complete in TMEM before it is read as the A operand
        if (!mbar_wait(bar(D1_DONE), ph, abort_flag)) break;
        if (!mbar_wait(bar(S_FULL), ph, abort_flag)) break;
        if (!mbar_wait(bar(ACC_FREE), ph ^ 1, abort_flag)) break;
        tc_fence_after();
        {
          const uint64_t dS = desc_kmajor(sbase + kOffS);
#pragma unroll
          for (uint32_t i = 0; i < 16; ++i)   // k chunk i >> 2 of the state, 8 values of k per step
            mma_tf32_ts(tmem + kColAcc, tmem + kColQf + i * 8, dS + (((i >> 2) * kTile + (i & 3u) * 32u) >> 4),
                        kIdTf32, i);
        }
        tc_commit(bar(S_FREE));
        // acc += [W ; A] V
        if (!mbar_wait(bar(V_FULL), ph, abort_flag)) break;
        tc_fence_after();
        {
          const uint64_t dW = desc_kmajor(sbase + kOffW), dVr = desc_mnmajor(sbase + kOffV, kTile);
#pragma unroll
          for (uint32_t i = 0; i < 8; ++i)   // 16 nodes j per step; hi then lo tile of [W ; A]
            mma_bf16_ss(tmem + kColAcc, dW + (((i & 1u) * kTile + (i >> 1) * 32u) >> 4),
                        dVr + (((i >> 1) * 2048u) >> 4), kIdMn, 1);
        }
        tc_commit(bar(V_FREE));
        tc_commit(bar(ACC_DONE));
      }
    }
  } else if (warp == kComputeWarps + 2) {
    if (lane == 0) {
      // ===================== output stores =====================
      // Staged chunks of item k leave by TMA; OST_FREE(k) tells the compute warps that the
      // chunks (which alias the Ak / W operand tiles) have been read and may be rewritten.
      uint32_t it = 0;
      for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++it) {
        if (!mbar_wait(bar(OST_READY), it & 1, abort_flag)) break;
        const Coord co = coord_of(item);
        if constexpr (PACKED) {
          // groups of 8 rows, largest boxes first (staging rows start on 1024-byte boundaries)
          const PackedItem pi = packed_item(p.offsets, p.B, p.H, p.Hk, item, p.div);
          const int full = pi.n & ~7;
          for (int part = 0; part < (want_U ? 2 : 1); ++part) {
            const OutMaps& mm = part == 0 ? mapsO : mapsU;
            int r = 0;
            auto put = [&](const CUtensorMap* m, int rows_box) {
              while (full - r >= rows_box) {
#pragma unroll
                for (int c = 0; c < 4; ++c)
                  store_box(m, sbase + kOffStage + (part * 4 + c) * 8192 + (uint32_t)r * 128u, nf_o, 32 * c,
                            co.y0 + r, co.h, co.z);
                r += rows_box;
              }
            };
            put(&mm.m64, 64);
            put(&mm.m32, 32);
            put(&mm.m16, 16);
            put(&mm.m8, 8);
          }
        } else {
#pragma unroll
          for (int c = 0; c < 4; ++c) store_box(&tmO, sbase + kOffStage + c * 8192, nf_o, 32 * c, 0, co.h, co.z);
          if (want_U) {
#pragma unroll
            for (int c = 0; c < 4; ++c) store_box(&tmU, sbase + kOffStage + (4 + c) * 8192, nf_o, 32 * c, 0, co.h, co.z);
          }
        }
        tma_store_commit();
        tma_store_wait_read();
        mbar_arrive(bar(OST_FREE));
      }
      tma_store_wait_all();
    }
  } else if (warp == kComputeWarps + 3) {
    // ===================== metadata warp =====================
    // Item j's strict-ancestor masks, alpha and beta go to buffer j & 1 while the compute
    // warps work on item j-1; the buffer is free once they have finished item j-2.
    grid_dependency_wait();   // tree metadata and gates may come from the kernels in front
    uint32_t j = 0;
    for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++j) {
      const uint32_t buf = j & 1, use = j >> 1;
      if (use > 0 && !mbar_wait_warp(bar(buf ? META_FREE1 : META_FREE), (use - 1) & 1, abort_flag)) break;
      int n = T, tb = 0;
      int64_t g0, gstep = 1;                            // first gate of the item, step between nodes
      if constexpr (PACKED) {
        const PackedItem pi = packed_item(p.offsets, p.B, p.H, p.Hk, item, p.div);
        n = pi.n;
        tb = pi.b;
        g0 = (int64_t)pi.plane_v * p.capacity + pi.row0;
      } else {
        const int lb = (int)fdiv((uint32_t)item, p.div.dH);
        tb = p.tree.n_trees == 1 ? 0 : request_of(item, p.B, p.div);
        g0 = (int64_t)lb * p.gate.b + (int64_t)(item - lb * p.H) * p.gate.h;
        gstep = p.gate.t;
      }
      float* tab = tab_s + buf * (2 * kRows);
      // all six loads first: one trip to memory, not one per table
      uint64_t mk[2] = {0ull, 0ull};
      float al[2] = {1.f, 1.f}, be[2] = {0.f, 0.f};
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int nd = lane + 32 * h;
        if (nd < n) {
          mk[h] = __ldg(reinterpret_cast<const unsigned long long*>(p.tree.anc) + ((size_t)tb * T + nd) * 2);
          al[h] = __ldg(p.alpha + g0 + nd * gstep);
          be[h] = __ldg(p.beta + g0 + nd * gstep);
        }
      }
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int nd = lane + 32 * h;
        mask_s[buf * kRows + nd] = mk[h];
        tab[nd] = al[h];
        tab[kRows + nd] = be[h];
        // the node's path in slot order: the set bits of (ancestors | self) from the lowest up
        // (nodes are numbered parent before child); slots past the node's depth are never used
        uint8_t* prow = Ps_all + (buf * kRows + nd) * kLdP;
        uint64_t rest = nd < n ? (mk[h] | (1ull << nd)) : 0ull;
        for (int s2 = 0; rest != 0ull && s2 < kSlots; ++s2) {
          prow[s2] = (uint8_t)(__ffsll((long long)rest) - 1);
          rest &= rest - 1;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(buf ? META_FULL1 : META_FULL));
    }
  } else {
    // ===================== compute warps =====================
    const int cw = warp - 2;
    const int quad = warp & 3;
    const int hc = cw >> 2;                 // which of the two threads of a row
    const int row = quad * 32 + lane;       // tile row
    const int node = row & 63;              // tree node of this row
    const int part = row >> 6;              // 0: O problem, 1: U problem
    const bool rows_live = (quad & 1) * 32 < T;                  // warp-uniform: some row of the warp is a node
    const bool live = node < T && (part == 0 || want_U);         // this row carries a problem
    const bool warp_live = rows_live && (part == 0 || want_U);   // same, for the warp-wide tcgen05.ld/st
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t swz = (uint32_t)(row & 7);
    const uint32_t nswz = (uint32_t)(node & 7);

    // Ancestor masks, alpha and beta of every item are put into shared memory by the
    // metadata warp, one item ahead (META_FULL / META_FREE, two buffers).
    PackedItem npk = {0, 0, 0, 0, T};   // packed forest: rows of the next item
    auto next_rows = [&](int item) {
      if constexpr (PACKED) {
        if (item < p.n_items) npk = packed_item(p.offsets, p.B, p.H, p.Hk, item, p.div);
      }
    };
    grid_dependency_wait();   // tree metadata comes from the kernel in front (dependent launch)
    // the commit kernel behind this one may be scheduled as SMs drain (it orders itself)
    if (warp == 2 && lane == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    next_rows(blockIdx.x);

    // acc rows 0..63 -> O chunks 0..3, rows 64..127 -> U chunks 4..7 (the chunks alias the Ak / W
    // tiles, which are idle between the readout MMA of item k and E2 of item k+1)
    auto final_epilogue = [&](uint32_t it_prev, const PackedItem& pk_prev) -> bool {
      if (!mbar_wait_warp(bar(ACC_DONE), it_prev & 1, abort_flag)) return false;
      tc_fence_after();
      if (warp_live) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t r1[32];
          tmem_ld32(tmem + lane_addr + kColAcc + hc * 64 + half * 32, r1);
          tmem_wait_ld();
          unsigned char* orow = sm + kOffStage + (part * 4 + hc * 2 + half) * 8192 + node * 128;
          // packed forest: the rows after the last full group of 8 leave from registers
          const bool tail_row = PACKED && node >= (pk_prev.n & ~7) && node < pk_prev.n;
          float* otail = nullptr;
          if constexpr (PACKED)
            otail = (part == 0 ? p.O : p.U) +
                    ((size_t)pk_prev.plane_v * p.capacity + pk_prev.row0 + node) * 128 + hc * 64 + half * 32;
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            const uint4 o4 = make_uint4(r1[4 * c], r1[4 * c + 1], r1[4 * c + 2], r1[4 * c + 3]);
            *reinterpret_cast<uint4*>(orow + (((uint32_t)c ^ nswz) << 4)) = o4;
            if (tail_row) *reinterpret_cast<uint4*>(otail + 4 * c) = o4;
          }
        }
      }
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar(ACC_FREE));
        mbar_arrive(bar(OST_READY));
      }
      return true;
    };

    uint32_t it = 0;
    bool ok = true;
    PackedItem pk = npk, pk_prev = npk;
    const int total_rows = PACKED ? p.offsets[p.B] : 0;   // rows at and past this one hold no node
    // One pass more than the CTA has items: the last one only writes out the last item (the
    // output code exists once).
#pragma unroll 1
    for (int item = blockIdx.x;; item += gridDim.x, ++it) {
      const bool item_live = item < p.n_items;
      const uint32_t ph = it & 1;
      pk = npk;
      const int Tb = PACKED ? pk.n : T;                       // real nodes of this item
      const bool live_i = live && node < Tb && item_live;
      constexpr int NS = DMAX + 1;                            // path slots in use
      int path[NS];
      float al[NS], bt[NS], pre[NS], vec[NS];
      float Pi = 1.f;                                         // P_i: product of alpha along the path
      int depth = 0;
      if (item_live) {
      // Every warp has finished the row solve of the previous item (it read the slot tables and
      // the per-node tables that this item is about to overwrite; with the Gram product issued one
      // item ahead, nothing else would hold a fast warp back).
      if (it > 0 && !(ok = mbar_wait_warp(bar(W_READY), (it - 1) & 1, abort_flag))) break;
      // ---- per-node tables of this item (written by the metadata warp) ----
      if (!(ok = mbar_wait_warp(bar(ph ? META_FULL1 : META_FULL), (it >> 1) & 1, abort_flag))) break;
      const uint64_t m = node < Tb ? mask_s[ph * kRows + node] : 0ull;   // strict ancestors
      const float* al_s = tab_s + ph * (2 * kRows);
      const float* be_s = al_s + kRows;
      next_rows(item + (int)gridDim.x);
      depth = __popcll(m);

      // ---- E1: raw path-sparse rows: part 0 <- Q K^T (path incl. the node), part 1 <- K K^T ----
      if (!(ok = mbar_wait_warp(bar(G_DONE), ph, abort_flag))) break;
      tc_fence_after();
      // A node's ancestors have smaller numbers than the node: the rows of nodes 0..31 select
      // nothing among the columns 32..63, and the warp that would scan them skips the chunk.
      if (rows_live && !(hc == 1 && (quad & 1) == 0)) {
        const uint64_t sel = node < Tb ? (part == 0 ? (m | (1ull << node)) : m) : 0ull;
        float* dst = (part == 0 ? Cs : Gs) + node * kLd;
        const int cbase = hc * 32;
        const uint32_t bits = (uint32_t)(sel >> cbase);
        const int base = hc ? __popc((uint32_t)sel) : 0;      // slots taken by columns 0..31
        uint32_t r[32];
        tmem_ld32(tmem + lane_addr + kColSc + cbase, r);
        tmem_wait_ld();
#pragma unroll
        for (int jj = 0; jj < 32; ++jj) {
          // unselected columns land in the padding slot of the row: no branch, no predicate
          // (predicated stores of the selected columns only were measured slower)
          const int slot = ((bits >> jj) & 1u) ? base + __popc(bits & ((1u << jj) - 1u)) : kSlots;
          dst[slot] = __uint_as_float(r[jj]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar(G_FREE));
        mbar_arrive(bar(E1_SYNC));
      }
      if (!(ok = mbar_wait_warp(bar(E1_SYNC), ph, abort_flag))) break;

      // ---- E2: decay factors, one back-substitution per row, operand tiles ----
      if (live_i) {
        const uint32_t* pw = reinterpret_cast<const uint32_t*>(Ps_all + (ph * kRows + node) * kLdP);
        const uint32_t pword[4] = {pw[0], pw[1], pw[2], pw[3]};
#pragma unroll
        for (int s2 = 0; s2 < NS; ++s2) {
          path[s2] = (pword[s2 >> 2] >> ((s2 & 3) * 8)) & 63;
          const bool on = s2 <= depth;
          const float a2 = al_s[path[s2]], b2 = be_s[path[s2]];
          al[s2] = on ? a2 : 1.f;    // slots past the node count as no decay
          bt[s2] = on ? b2 : 0.f;
          Pi *= al[s2];
          pre[s2] = Pi;              // P at path node s2
        }
      }
      // ---- output of the previous item: its MMAs ran under E1 and the gather above, so the
      // accumulator is complete by now; the TMA stores that take the staged chunks away read them
      // under the back-substitution and the Qf initialisation below ----
      }
      if (it > 0 && !(ok = final_epilogue(it - 1, pk_prev))) break;
      if (!item_live) break;
      if (live_i) {
        // C_{i,p_s} = (q_i . k_{p_s}) P_i / P_{p_s}: the ratio is the product of alpha over the
        // slots after s, built up from the node's own slot backwards
        float sfx = 1.f;
#pragma unroll
        for (int s2 = NS - 1; s2 >= 0; --s2) {
          const float c = Cs[node * kLd + s2];
          if (part == 0) vec[s2] = s2 <= depth ? c * sfx : 0.f;
          else vec[s2] = s2 == depth ? 1.f : 0.f;                               // x L = e_d
          sfx *= al[s2];
        }
        // w_s = c_s - sum_{t > s} w_t G_{p_t,p_s},  G_{p_t,p_s} = beta_t (P_{p_t} / P_{p_s}) k_t.k_s;
        // rr[t] holds P_{p_t} / P_{p_s} = alpha_{s+1} ... alpha_t for the current s and grows by one
        // factor per step.  Slots past the node's depth carry vec = 0 and a deselected G, so nothing
        // is predicated.
        float rr[NS];
#pragma unroll
        for (int s2 = NS - 2; s2 >= 0; --s2) {
          float acc = vec[s2];
#pragma unroll
          for (int t = s2 + 1; t < NS; ++t) {
            rr[t] = t == s2 + 1 ? al[t] : rr[t] * al[s2 + 1];
            const float gts = Gs[path[t] * kLd + s2] * (bt[t] * rr[t]);
            acc = fmaf(-vec[t], t <= depth ? gts : 0.f, acc);
          }
          if (s2 < depth) vec[s2] = acc;
        }
      }
      // Qf starts as D_P Q (rows of the O problem; P_i in full fp32) or 0 (rows of the U problem):
      // the key-product MMA accumulates -(W D_P) K on top.  The state MMA of the previous item
      // must have read the old Qf first.
      if (it > 0 && !(ok = mbar_wait_warp(bar(S_FREE), (it - 1) & 1, abort_flag))) break;
      // the Q rows are read by these threads: observe the load's barrier themselves
      if (!(ok = mbar_wait_warp(bar((it & 1) ? QK_FULL1 : QK_FULL), (it >> 1) & 1, abort_flag))) break;
      if (warp_live) {
        const bool use_q = live_i && part == 0;
        const float Pq = Pi * kTf32Comp;
        const unsigned char* qrow = sm + ((it & 1) ? kOffQK1 : kOffQK) + hc * kTile + node * 128;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t r[32];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const uint4 x = *reinterpret_cast<const uint4*>(qrow + (((uint32_t)(half * 4 + c) ^ nswz) << 4));
            const uint32_t w4[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              // select, never 0 * x: rows past the request may hold anything
              r[c * 8 + 2 * e] = use_q ? __float_as_uint(Pq * __uint_as_float(w4[e] << 16)) : 0u;
              r[c * 8 + 2 * e + 1] = use_q ? __float_as_uint(Pq * __uint_as_float(w4[e] & 0xffff0000u)) : 0u;
            }
          }
          tmem_st32(tmem + lane_addr + kColQf + hc * 64 + half * 32, r);
        }
        tmem_wait_st();
      }
      // The tiles alias the staged output chunks of the previous item: its stores must have read
      // them (they did so under the Qf initialisation above).
      if (it > 0 && !(ok = mbar_wait_warp(bar(OST_FREE), (it - 1) & 1, abort_flag))) break;
      if constexpr (PACKED) {
        // A box that reaches past the last node of the forest brings rows nobody wrote.  They only
        // ever meet zero coefficients, but 0 x garbage need not be 0: zero them.  The Gram MMA has
        // finished with Q and K (G_DONE above); V is waited for here.
        if (pk.row0 + kRows > total_rows) {
          if (!(ok = mbar_wait_warp(bar(V_FULL), ph, abort_flag))) break;
          if (node >= total_rows - pk.row0 && !(part == 1 && hc == 1)) {
            const uint32_t qk_base = (it & 1) ? kOffQK1 : kOffQK;
            const uint32_t base = part == 1 ? kOffV : hc == 0 ? qk_base : qk_base + 8192;
            const uint4 z = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int tile = 0; tile < 2; ++tile)
#pragma unroll
              for (int c = 0; c < 8; ++c)
                *reinterpret_cast<uint4*>(sm + base + tile * kTile + node * 128 + c * 16) = z;
          }
        }
      }
      if (live_i) {
        // hc 0 writes the [W ; A] tiles, hc 1 the -[W D_P ; A D_P] tiles
        unsigned char* trow = sm + (hc == 0 ? kOffW : kOffAk) + row * 128;
        const uint4 z = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int tile = 0; tile < 2; ++tile)
#pragma unroll
          for (int c = 0; c < 8; ++c)
            *reinterpret_cast<uint4*>(trow + tile * kTile + (((uint32_t)c ^ swz) << 4)) = z;
#pragma unroll
        for (int s2 = 0; s2 < NS; ++s2) {
          if (s2 <= depth) {
            const int j = path[s2];
            const float wv = vec[s2] * bt[s2];                        // W = C N D_beta (or A = N D_beta)
            const float val = hc == 0 ? wv : -(wv * pre[s2]) * kTf32Comp;   // ... times P_{p_s}, negated
            const uint32_t off = ((((uint32_t)j >> 3) ^ swz) << 4) + ((uint32_t)j & 7u) * 2u;
            uint16_t hi, lo;
            split_bf16(val, hi, lo);
            *reinterpret_cast<uint16_t*>(trow + off) = hi;
            *reinterpret_cast<uint16_t*>(trow + kTile + off) = lo;
          }
        }
      }
      tc_fence_before();
      fence_async_smem();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar(W_READY));
        mbar_arrive(bar(ph ? META_FREE1 : META_FREE));   // this item's tables may be overwritten
      }
      pk_prev = pk;
    }
  }

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u)
                 : "memory");
  }
  if (tid == 0 && *abort_flag && p.status) atomicExch(p.status, (int)TV_ERR_DEVICE_TIMEOUT);
}

}  // namespace

bool tv_verify_tc_delta_supports(const VerifyArgs& a) {
  return a.bf16 && a.dk == 128 && a.dv == 128 && a.rule == TV_GATED_DELTA && a.T <= kRows &&
         a.tree.max_depth_all < kSlots;
}

int tv_launch_verify_tc_delta(const VerifyArgs& a, int32_t* status, cudaStream_t stream) {
  if (!tv_verify_tc_delta_supports(a)) return TV_ERR_UNSUPPORTED;
  const bool packed = a.tree.offsets != nullptr;
  const uint64_t items = (uint64_t)a.L * a.B * a.H;
  // the U maps are only used when U is requested; O stands in otherwise
  float* Uout = a.U ? a.U : a.O;
  const void* const ptrs[5] = {a.q, a.k, a.v, a.S_pre, a.O};
  const void* const uptrs[5] = {Uout, nullptr, nullptr, nullptr, nullptr};
  // 4-D views: dense / strided layouts from the resolved strides, packed forests as planes
  NodeView vq, vv, vo;
  if (!packed) {
    const uint64_t lb = (uint64_t)a.L * a.B;
    vq = NodeView{128, (uint64_t)a.T, (uint64_t)a.Hk, lb, a.lay.qk.b, a.lay.qk.h, a.lay.qk.t};
    vv = NodeView{128, (uint64_t)a.T, (uint64_t)a.H, lb, a.lay.v.b, a.lay.v.h, a.lay.v.t};
    vo = NodeView{128, (uint64_t)a.T, (uint64_t)a.H, lb, a.lay.out.b, a.lay.out.h, a.lay.out.t};
  } else {
    const int64_t cap = a.tree.capacity;
    vq = NodeView{128, (uint64_t)cap, (uint64_t)a.Hk, (uint64_t)a.L, (int64_t)a.Hk * cap * 128, cap * 128, 128};
    vv = NodeView{128, (uint64_t)cap, (uint64_t)a.H, (uint64_t)a.L, (int64_t)a.H * cap * 128, cap * 128, 128};
    vo = vv;
  }
  const uint64_t key = view_key(vq) * 3 + view_key(vv) * 5 + view_key(vo) * 7 + items;
  const MapSet* ms = nullptr;   // q, k, v, S, O (64-row boxes)
  const MapSet* mu = nullptr;   // U (64-row boxes)
  const MapSet* mo2 = nullptr;  // packed forest: O boxes of 32, 16, 8 rows
  const MapSet* mu2 = nullptr;  // packed forest: U boxes of 32, 16, 8 rows
  ms = cached_maps(ptrs, key, a.T, (packed ? 6 : 1) | (a.Hk << 8), [&](CUtensorMap* m) {
    return make_map4(&m[0], a.q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, vq, 64, 64) &&
           make_map4(&m[1], a.k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, vq, 64, 64) &&
           make_map4(&m[2], a.v, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, vv, 64, 64) &&
           make_map(&m[3], a.S_pre, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, items, 128, 128, 32, 128) &&
           make_map4(&m[4], a.O, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, vo, 32, 64);
  });
  if (!packed) {
    mu = cached_maps(uptrs, key, a.T, 2, [&](CUtensorMap* m) {
      return make_map4(&m[0], Uout, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, vo, 32, 64);
    });
  } else {
    auto small_boxes = [&](float* base) {
      return [=](CUtensorMap* m) {
        return make_map4(&m[0], base, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, vo, 32, 32) &&
               make_map4(&m[1], base, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, vo, 32, 16) &&
               make_map4(&m[2], base, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, vo, 32, 8) &&
               make_map4(&m[3], base, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, vo, 32, 64);
      };
    };
    const void* const optrs[5] = {a.O, nullptr, nullptr, nullptr, (const void*)1};
    const void* const u2ptrs[5] = {Uout, nullptr, nullptr, nullptr, (const void*)2};
    mo2 = cached_maps(optrs, key, a.T, 7, small_boxes(a.O));
    mu2 = cached_maps(u2ptrs, key, a.T, 7, small_boxes(Uout));
    mu = mu2;
  }
  if (!ms || !mu || (packed && (!mo2 || !mu2))) return TV_ERR_CUDA;
  OutMaps mapsO, mapsU;
  if (packed) {
    mapsO.m64 = ms->map[4]; mapsO.m32 = mo2->map[0]; mapsO.m16 = mo2->map[1]; mapsO.m8 = mo2->map[2];
    mapsU.m64 = mu2->map[3]; mapsU.m32 = mu2->map[0]; mapsU.m16 = mu2->map[1]; mapsU.m8 = mu2->map[2];
  } else {
    mapsO.m64 = mapsO.m32 = mapsO.m16 = mapsO.m8 = ms->map[4];
    mapsU.m64 = mapsU.m32 = mapsU.m16 = mapsU.m8 = mu->map[0];
  }
  static thread_local int configured_dev = -1;
  static thread_local int sm_count = 0;
  int dev = 0;
  TV_CUDA_TRY(cudaGetDevice(&dev));
  if (configured_dev != dev) {
    TV_CUDA_TRY(cudaFuncSetAttribute(verify_tc_delta_kernel<8, false>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
    TV_CUDA_TRY(cudaFuncSetAttribute(verify_tc_delta_kernel<15, false>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
    TV_CUDA_TRY(cudaFuncSetAttribute(verify_tc_delta_kernel<8, true>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
    TV_CUDA_TRY(cudaFuncSetAttribute(verify_tc_delta_kernel<15, true>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
    TV_CUDA_TRY(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev));
    configured_dev = dev;
  }
  DeltaParams p;
  p.tree = a.tree;
  p.n_items = (int32_t)items;
  p.B = a.B; p.H = a.H; p.T = a.T; p.Hk = a.Hk;
  p.alpha = a.alpha;
  p.beta = a.beta;
  p.want_U = a.U != nullptr;
  p.status = status;
  p.offsets = a.tree.offsets;
  p.capacity = a.tree.capacity;
  p.div = make_item_div(a.B, a.H, a.Hk);
  p.gate = a.lay.gate;
  p.node_first = (node_first_of(vq) ? 1 : 0) | (node_first_of(vv) ? 2 : 0) | (node_first_of(vo) ? 4 : 0);
  p.O = a.O;
  p.U = Uout;
  // With a few items per CTA, as many CTAs as give every one the same number of items (512 items
  // on 148 SMs: 128 CTAs of 4 rather than 148 of 3 or 4 -- the launch takes four item periods
  // either way, and the CTAs that run share the memory system with fewer others: 43.1 -> 42.6 us
  // per step on that workload).  With many items per CTA an idle SM costs more than the balance
  // gains (the gated kernel on 28 items per CTA: 0.8 % slower), so the rule stops at eight.
  int grid = (int)(items < (uint64_t)sm_count ? items : (uint64_t)sm_count);
  if (items > (uint64_t)sm_count) {
    const uint64_t rounds = (items + sm_count - 1) / sm_count;
    if (rounds <= 8) grid = (int)((items + rounds - 1) / rounds);
  }
  const bool shallow = a.tree.max_depth_all <= 8;
  auto launch = [&](auto kernel) {
    return launch_dependent(kernel, grid, kThreads, kSmemBytes, stream, ms->map[0], ms->map[1], ms->map[2],
                            ms->map[3], mapsO, mapsU, p);
  };
  if (packed)
    TV_CUDA_TRY(shallow ? launch(verify_tc_delta_kernel<8, true>) : launch(verify_tc_delta_kernel<15, true>));
  else
    TV_CUDA_TRY(shallow ? launch(verify_tc_delta_kernel<8, false>) : launch(verify_tc_delta_kernel<15, false>));
  TV_CUDA_TRY(cudaGetLastError());
  return TV_OK;
}
