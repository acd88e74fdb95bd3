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
// FMAs per row, no T x T product, no Neumann rounds, no level barriers.
//
// Tile rows 0..63 carry the O problem of node i, rows 64..127 the U problem of
// node i (the M = 128 MMA shape is otherwise half empty at T <= 64):
//     Sc1 = Q K^T, Sc2 = K K^T                 (bf16, N = 64)        -> TMEM
//     rows of [W ; A] and [W D_P ; A D_P]      (fp32 threads)        -> bf16 hi/lo tiles
//     D1  = [W D_P ; A D_P] K                  (bf16, K as MN-major B)
//     Qf  = [D_P Q - D1 ; -D1]                 (fp32 -> TMEM, tf32 A operand)
//     acc = Qf S_pre^T + [W ; A] V             (tf32 + bf16 hi/lo)
//     O = acc[0..63], U = acc[64..127]
// S_pre goes TMA -> shared memory -> tensor core untouched; O leaves through
// swizzled staging tiles and a TMA store.  Every wait is a bounded mbarrier
// wait (status word on expiry); no TMA multicast.
#include "tv_tc_common.cuh"

namespace {

using namespace tvtc;

constexpr int kThreads = 320;
constexpr int kComputeWarps = 8;
constexpr int kSlots = 16;     // path slots per node: depth <= 15
constexpr int kRows = 64;      // T <= 64

// shared memory map (bytes from the 1024-aligned base); operand tiles are 128 x 128 B,
// TMA fills rows 0..63 only; the upper halves (rows 64..127) hold scratch and staging
constexpr uint32_t kOffQ = 0;                    // 2 k-halves of Q; upper halves: O staging 0,1
constexpr uint32_t kOffK = 2 * kTile;            // 2 k-halves of K; upper halves: O staging 2,3
constexpr uint32_t kOffV = 4 * kTile;            // 2 dv-halves of V; upper halves: scratch
constexpr uint32_t kOffS = 6 * kTile;            // 4 k-chunks of S_pre [128 v][32] f32
constexpr uint32_t kOffW = 10 * kTile;           // [W;A] hi, lo, [W D_P;A D_P] hi, lo: [128][64] bf16
constexpr int kLd = 17;                          // row stride of the slot tables (floats): no bank
                                                 // conflict when 32 nodes touch the same slot
constexpr int kLdP = 20;                         // row stride of the path table (bytes)
constexpr uint32_t kOffGs = kOffV + 8192;        // float Gs[64][kLd]: G_{i,p_s}
constexpr uint32_t kOffCs = kOffV + kTile + 8192;  // float Cs[64][kLd]: C_{i,p_s}
constexpr uint32_t kOffPs = kOffCs + 4352;       // uint8 Ps[64][kLdP]: path nodes
constexpr uint32_t kOffSmall = kOffPs + 1280;    // float g, f, la, be, P [64] each
constexpr uint32_t kOffBar = 14 * kTile;
constexpr uint32_t kOffMisc = kOffBar + 8 * 24;
constexpr uint32_t kSmemBytes = kOffMisc + 64 + 1024;

enum Bar {
  QK_FULL = 0, QK_FREE, S_FULL, S_FREE, V_FULL, V_FREE,
  G_DONE, G_FREE, W_READY, D1_DONE, QF_READY, ACC_DONE, ACC_FREE, SETUP, E1_SYNC,
  OST_READY, OST_FREE
};

constexpr uint32_t kColQf = 0, kColSc1 = 128, kColSc2 = 192, kColD1 = 256, kColAcc = 384;

// Phase timestamps for kernel tuning: compiled out unless TV_TC_PROFILE is defined.
#ifdef TV_TC_PROFILE
__device__ long long* g_tcd_prof = nullptr;
#define TCD_STAMP(it, slot)                                                       \
  do {                                                                            \
    if (g_tcd_prof && blockIdx.x == 0 && (it) < 16 && lane == 0)                  \
      g_tcd_prof[(it) * 32 + (slot)] = clock64();                                 \
  } while (0)
#else
#define TCD_STAMP(it, slot) do { } while (0)
#endif

struct DeltaParams {
  TreeDev tree;
  int32_t n_items, B, H, T;
  const float* alpha;
  const float* beta;
  float* U;        // [items][T][128] or nullptr
  int32_t* status;
};

// fp32 -> tf32 with round-to-nearest (the tensor core would otherwise cut the low 13 bits)
__device__ __forceinline__ uint32_t to_tf32_rn(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return r;
}

// bf16 hi/lo parts of x (hi = upper 16 bits, lo = upper 16 bits of the exact remainder)
__device__ __forceinline__ void split_bf16(float x, uint16_t& hi, uint16_t& lo) {
  const uint32_t b = __float_as_uint(x);
  const uint32_t h = b & 0xffff0000u;
  hi = (uint16_t)(h >> 16);
  lo = (uint16_t)(__float_as_uint(x - __uint_as_float(h)) >> 16);
}

__global__ void __launch_bounds__(kThreads, 1)
verify_tc_delta_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmS,
                       const __grid_constant__ CUtensorMap tmO, const DeltaParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(sm);
  float* Gs = reinterpret_cast<float*>(sm + kOffGs);
  float* Cs = reinterpret_cast<float*>(sm + kOffCs);
  uint8_t* Ps = reinterpret_cast<uint8_t*>(sm + kOffPs);
  float* g_s = reinterpret_cast<float*>(sm + kOffSmall);
  float* f_s = g_s + kRows;
  float* la_s = f_s + kRows;
  float* be_s = la_s + kRows;
  float* P_s = be_s + kRows;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + kOffMisc + 4);
  volatile int* range_ok_s = reinterpret_cast<volatile int*>(sm + kOffMisc + 16);
  auto bar = [&](int i) { return sbase + kOffBar + 8u * i; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int T = p.T;
  const bool want_U = p.U != nullptr;
  const int dmax = p.tree.max_depth_all;   // <= 15, the same for every thread

  if (tid == 0) {
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    mbar_init(bar(QK_FULL), 1);  mbar_init(bar(QK_FREE), 1 + kComputeWarps);
    mbar_init(bar(S_FULL), 1);   mbar_init(bar(S_FREE), 1);
    mbar_init(bar(V_FULL), 1);   mbar_init(bar(V_FREE), 1);
    mbar_init(bar(G_DONE), 1);   mbar_init(bar(G_FREE), kComputeWarps);
    mbar_init(bar(W_READY), kComputeWarps);
    mbar_init(bar(D1_DONE), 1);
    mbar_init(bar(QF_READY), kComputeWarps);
    mbar_init(bar(ACC_DONE), 1); mbar_init(bar(ACC_FREE), kComputeWarps);
    mbar_init(bar(SETUP), kComputeWarps);
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
    // ===================== TMA producer =====================
    if (lane == 0) {
      int pend_qk = 0, pend_s = 0, pend_v = 0;
      uint32_t it = 0;
      for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++it) {
        const uint32_t ph = it & 1;
        if (!mbar_wait(bar(QK_FREE), ph ^ 1, abort_flag)) break;
        mbar_expect_tx(bar(QK_FULL), 4 * 8192);
        tma_load_3d(sbase + kOffQ, &tmQ, bar(QK_FULL), 0, 0, item);
        tma_load_3d(sbase + kOffQ + kTile, &tmQ, bar(QK_FULL), 64, 0, item);
        tma_load_3d(sbase + kOffK, &tmK, bar(QK_FULL), 0, 0, item);
        tma_load_3d(sbase + kOffK + kTile, &tmK, bar(QK_FULL), 64, 0, item);
        pend_qk = 1 + (int)ph;
        if (!mbar_wait(bar(S_FREE), ph ^ 1, abort_flag)) break;
        mbar_expect_tx(bar(S_FULL), 4 * kTile);
#pragma unroll
        for (int c = 0; c < 4; ++c)
          tma_load_3d(sbase + kOffS + c * kTile, &tmS, bar(S_FULL), 32 * c, 0, item);
        pend_s = 1 + (int)ph;
        if (!mbar_wait(bar(V_FREE), ph ^ 1, abort_flag)) break;
        mbar_expect_tx(bar(V_FULL), 2 * 8192);
        tma_load_3d(sbase + kOffV, &tmV, bar(V_FULL), 0, 0, item);
        tma_load_3d(sbase + kOffV + kTile, &tmV, bar(V_FULL), 64, 0, item);
        pend_v = 1 + (int)ph;
      }
      if (*abort_flag) {
        if (pend_qk) mbar_wait(bar(QK_FULL), pend_qk - 1, abort_flag + 1);
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
      uint32_t it = 0;
      for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++it) {
        const uint32_t ph = it & 1;
        // Gram tiles: Sc1 = Q K^T, Sc2 = K K^T (N = 64: only nodes j < 64 exist)
        if (!mbar_wait(bar(QK_FULL), ph, abort_flag)) break;
        TCD_STAMP(it, 4);
        if (!mbar_wait(bar(G_FREE), ph ^ 1, abort_flag)) break;
        tc_fence_after();
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int s = 0; s < 4; ++s) {
            const uint64_t kd = desc_kmajor(sbase + kOffK + h * kTile + s * 32);
            mma_bf16_ss(tmem + kColSc1, desc_kmajor(sbase + kOffQ + h * kTile + s * 32), kd, kIdGram,
                        (h | s) != 0);
            mma_bf16_ss(tmem + kColSc2, kd, kd, kIdGram, (h | s) != 0);
          }
        tc_commit(bar(G_DONE));
        // D1 = [W D_P ; A D_P] K   (A operand: hi/lo tiles, K extent 64; B: K tiles, MN-major)
        if (!mbar_wait(bar(W_READY), ph, abort_flag)) break;
        TCD_STAMP(it, 5);
        tc_fence_after();
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          const uint64_t bdesc = desc_mnmajor(sbase + kOffK + s * 2048, kTile);
          mma_bf16_ss(tmem + kColD1, desc_kmajor(sbase + kOffW + 2 * kTile + s * 32), bdesc, kIdMn, s != 0);
          mma_bf16_ss(tmem + kColD1, desc_kmajor(sbase + kOffW + 3 * kTile + s * 32), bdesc, kIdMn, 1);
        }
        tc_commit(bar(D1_DONE));
        tc_commit(bar(QK_FREE));
        // acc = Qf S_pre^T
        if (!mbar_wait(bar(S_FULL), ph, abort_flag)) break;
        TCD_STAMP(it, 6);
        if (!mbar_wait(bar(QF_READY), ph, abort_flag)) break;
        TCD_STAMP(it, 7);
        if (!mbar_wait(bar(ACC_FREE), ph ^ 1, abort_flag)) break;
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int s = 0; s < 4; ++s)
            mma_tf32_ts(tmem + kColAcc, tmem + kColQf + c * 32 + s * 8,
                        desc_kmajor(sbase + kOffS + c * kTile + s * 32), kIdTf32, (c | s) != 0);
        tc_commit(bar(S_FREE));
        // acc += [W ; A] V
        if (!mbar_wait(bar(V_FULL), ph, abort_flag)) break;
        TCD_STAMP(it, 8);
        tc_fence_after();
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          const uint64_t bdesc = desc_mnmajor(sbase + kOffV + s * 2048, kTile);
          mma_bf16_ss(tmem + kColAcc, desc_kmajor(sbase + kOffW + s * 32), bdesc, kIdMn, 1);
          mma_bf16_ss(tmem + kColAcc, desc_kmajor(sbase + kOffW + kTile + s * 32), bdesc, kIdMn, 1);
        }
        tc_commit(bar(V_FREE));
        tc_commit(bar(ACC_DONE));
        TCD_STAMP(it, 9);
      }
    }
  } else {
    // ===================== compute warps =====================
    const int cw = warp - 2;
    const int quad = warp & 3;
    const int hc = cw >> 2;                 // column half handled by this warp
    const int row = quad * 32 + lane;       // tile row
    const int node = row & 63;              // tree node of this row
    const int part = row >> 6;              // 0: O problem, 1: U problem
    const bool live = node < T && (part == 0 || want_U);             // this row carries a problem
    const bool warp_live = (quad & 1) * 32 < T && (part == 0 || want_U);   // same for the whole warp: the
                                                                     // tcgen05.ld/st below are warp-wide
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t swz = (uint32_t)(row & 7);

    uint64_t nm = 0;
    float nal = 1.f, nbe = 0.f;
    auto fetch_meta = [&](int item) {
      nm = 0; nal = 1.f; nbe = 0.f;
      if (item < p.n_items && node < T) {
        const int b = (item / p.H) % p.B;
        const int tb = p.tree.n_trees == 1 ? 0 : b;
        nm = p.tree.anc[((size_t)tb * T + node) * 2];
        nal = p.alpha[(size_t)item * T + node];
        nbe = p.beta[(size_t)item * T + node];
      }
    };
    fetch_meta(blockIdx.x);

    // Output of the previous item: acc rows 0..63 -> O (staging tiles + TMA store),
    // rows 64..127 -> U (plain stores, off the critical path).
    auto final_epilogue = [&](uint32_t it_prev, int item_prev) -> bool {
      if (warp == 2 && lane == 0) {
        tma_store_wait_read();            // the store of the item before has read the staging tiles
        mbar_arrive(bar(OST_FREE));
      }
      if (!mbar_wait_warp(bar(ACC_DONE), it_prev & 1, abort_flag)) return false;
      if (!mbar_wait_warp(bar(OST_FREE), it_prev & 1, abort_flag)) return false;
      tc_fence_after();
      if (warp_live) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t r1[32];
          tmem_ld32(tmem + lane_addr + kColAcc + hc * 64 + half * 32, r1);
          tmem_wait_ld();
          if (!live) continue;
          if (part == 0) {
            const int c4 = hc * 2 + half;   // 32-column chunk -> upper half of Q0, Q1, K0, K1 tiles
            unsigned char* orow = sm + kOffQ + c4 * kTile + 8192 + node * 128;
#pragma unroll
            for (int c = 0; c < 8; ++c)
              *reinterpret_cast<uint4*>(orow + (((uint32_t)c ^ swz) << 4)) =
                  make_uint4(r1[4 * c], r1[4 * c + 1], r1[4 * c + 2], r1[4 * c + 3]);
          } else {
            float* urow = p.U + ((size_t)item_prev * T + node) * 128 + hc * 64 + half * 32;
#pragma unroll
            for (int c = 0; c < 8; ++c)
              *reinterpret_cast<uint4*>(urow + 4 * c) =
                  make_uint4(r1[4 * c], r1[4 * c + 1], r1[4 * c + 2], r1[4 * c + 3]);
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
      if (warp == 2 && lane == 0) {
        if (mbar_wait(bar(OST_READY), it_prev & 1, abort_flag)) {
#pragma unroll
          for (int c = 0; c < 4; ++c)
            tma_store_3d(&tmO, sbase + kOffQ + c * kTile + 8192, 32 * c, 0, item_prev);
          tma_store_commit();
        }
      }
      return true;
    };

    uint32_t it = 0;
    bool ok = true;
    int item_prev = 0;
    for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++it) {
      const uint32_t ph = it & 1;
      if (warp == 4) TCD_STAMP(it, 16);
      const uint64_t m = nm;                                  // strict ancestors
      const float be = nbe;
      const float la_own = log2f(nal);
      const bool writer = part == 0 && hc == 0 && node < T;   // one thread per node fills the tables
      if (writer) { la_s[node] = la_own; be_s[node] = be; }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(SETUP));
      fetch_meta(item + (int)gridDim.x);
      if (!(ok = mbar_wait_warp(bar(SETUP), 0, abort_flag))) break;
      float g = 0.f;
      if (node < T) {
        g = la_own;
        uint64_t a0 = m;
        while (a0) { const int j = __ffsll((long long)a0) - 1; a0 &= a0 - 1; g += la_s[j]; }
      }
      const float Pi = exp2f(g);
      if (writer) { g_s[node] = g; f_s[node] = exp2f(-g); P_s[node] = Pi; }
      const bool range_ok_warp = __all_sync(0xffffffffu, node >= T || fabsf(g) <= 100.f);
      if (lane == 0) range_ok_s[cw] = range_ok_warp;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(SETUP));
      const int depth = __popcll(m);
      const uint64_t mplus = m | (1ull << node);

      // ---- E1: path-sparse rows of C (from Q K^T) and G (from K K^T) ----
      if (warp == 4) TCD_STAMP(it, 17);
      if (!(ok = mbar_wait_warp(bar(G_DONE), ph, abort_flag))) break;
      if (warp == 4) TCD_STAMP(it, 18);
      if (!(ok = mbar_wait_warp(bar(SETUP), 1, abort_flag))) break;
      tc_fence_after();
      bool fast = true;
#pragma unroll
      for (int w8 = 0; w8 < kComputeWarps; ++w8) fast = fast && range_ok_s[w8];
      if (part == 0 && warp_live) {
        const uint64_t sel = node < T ? (hc == 0 ? mplus : m) : 0ull;
        float* dst = (hc == 0 ? Cs : Gs) + node * kLd;
        const float lead = (hc == 0 ? 1.f : be) * (fast ? Pi : 1.f);
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          uint32_t r[32];
          tmem_ld32(tmem + lane_addr + (hc == 0 ? kColSc1 : kColSc2) + half * 32, r);
          tmem_wait_ld();
          const uint32_t bits = (uint32_t)(sel >> (half * 32));
          const int base = half ? __popc((uint32_t)sel) : 0;   // slots taken by columns 0..31
          // Every column is independent: its slot is the number of selected columns before it.
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4) {
            const float4 f4 = *reinterpret_cast<const float4*>((fast ? f_s : g_s) + half * 32 + q4 * 4);
            const float fv[4] = {f4.x, f4.y, f4.z, f4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int jj = q4 * 4 + e;
              const float ratio = fast ? fv[e] : exp2f(g - fv[e]);   // P_i / P_j (times P_i in `lead`)
              const float val = lead * ratio * __uint_as_float(r[jj]);
              // unselected columns land in the padding slot of the row: no branch, no predicate
              const int slot = ((bits >> jj) & 1u) ? base + __popc(bits & ((1u << jj) - 1u)) : kSlots;
              dst[slot] = val;
              if (hc == 0) Ps[node * kLdP + slot] = (uint8_t)(half * 32 + jj);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar(G_FREE));
        mbar_arrive(bar(E1_SYNC));
      }
      if (warp == 4) TCD_STAMP(it, 19);
      if (!(ok = mbar_wait_warp(bar(E1_SYNC), ph, abort_flag))) break;
      if (warp == 4) TCD_STAMP(it, 20);

      // ---- E2: one back-substitution per row on the path system, then the operand tiles ----
      if (hc == 0 && live) {
        // path nodes and the right-hand side into registers (16 slots, statically indexed)
        const uint32_t* pw = reinterpret_cast<const uint32_t*>(Ps + node * kLdP);
        const uint32_t pword[4] = {pw[0], pw[1], pw[2], pw[3]};
        int path[kSlots];
#pragma unroll
        for (int s2 = 0; s2 < kSlots; ++s2) path[s2] = (pword[s2 >> 2] >> ((s2 & 3) * 8)) & 0xff;
        float vec[kSlots];
        if (part == 0) {
#pragma unroll
          for (int s2 = 0; s2 < kSlots; ++s2) vec[s2] = s2 <= depth ? Cs[node * kLd + s2] : 0.f;
        } else {
#pragma unroll
          for (int s2 = 0; s2 < kSlots; ++s2) vec[s2] = s2 == depth ? 1.f : 0.f;   // x L = e_d
        }
        if (warp == 4) TCD_STAMP(it, 25);
        // w_s = c_s - sum_{t > s} w_t G_{p_t, p_s}, from the node upwards
#pragma unroll
        for (int s2 = kSlots - 2; s2 >= 0; --s2) {
          if (s2 < dmax) {                                    // CTA-uniform bound
            // slots past the node's depth hold vec = 0 and a deselected G: loads carry no predicate
            float acc = vec[s2];
#pragma unroll
            for (int t = s2 + 1; t < kSlots; ++t) {
              const float gts = Gs[(path[t] & 63) * kLd + s2];
              acc = fmaf(-vec[t], t <= depth ? gts : 0.f, acc);
            }
            if (s2 < depth) vec[s2] = acc;
          }
        }
        if (warp == 4) TCD_STAMP(it, 26);
        unsigned char* trow = sm + kOffW + row * 128;
        const uint4 z = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int tile = 0; tile < 4; ++tile)
#pragma unroll
          for (int c = 0; c < 8; ++c)
            *reinterpret_cast<uint4*>(trow + tile * kTile + (((uint32_t)c ^ swz) << 4)) = z;
        if (warp == 4) TCD_STAMP(it, 27);
#pragma unroll
        for (int s2 = 0; s2 < kSlots; ++s2) {
          if (s2 <= dmax && s2 <= depth) {
            const int j = path[s2];
            const float wv = vec[s2] * be_s[j];                // row of W = C N D_beta (or A = N D_beta)
            const float wp = wv * P_s[j];                      // row of W D_P (or A D_P)
            const uint32_t off = ((((uint32_t)j >> 3) ^ swz) << 4) + ((uint32_t)j & 7u) * 2u;
            uint16_t hi, lo;
            split_bf16(wv, hi, lo);
            *reinterpret_cast<uint16_t*>(trow + off) = hi;
            *reinterpret_cast<uint16_t*>(trow + kTile + off) = lo;
            split_bf16(wp, hi, lo);
            *reinterpret_cast<uint16_t*>(trow + 2 * kTile + off) = hi;
            *reinterpret_cast<uint16_t*>(trow + 3 * kTile + off) = lo;
          }
        }
      }
      if (warp == 4) TCD_STAMP(it, 28);
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(W_READY));
      if (warp == 4) TCD_STAMP(it, 21);

      // ---- output of the previous item, under the D1 MMA of this one ----
      if (it > 0 && !(ok = final_epilogue(it - 1, item_prev))) break;

      // ---- E3: Qf = [D_P Q - D1 ; -D1] -> TMEM (A operand of the state contraction) ----
      if (warp == 4) TCD_STAMP(it, 22);
      if (!(ok = mbar_wait_warp(bar(D1_DONE), ph, abort_flag))) break;
      if (warp == 4) TCD_STAMP(it, 23);
      tc_fence_after();
      if (warp_live) {
        const unsigned char* qrow = sm + kOffQ + hc * kTile + node * 128;
        const uint32_t qswz = (uint32_t)(node & 7);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t r[32];
          tmem_ld32(tmem + lane_addr + kColD1 + hc * 64 + half * 32, r);
          tmem_wait_ld();
          if (part == 0) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const uint4 x = *reinterpret_cast<const uint4*>(qrow + (((half * 4 + c) ^ qswz) << 4));
              const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                r[c * 8 + 2 * e] = to_tf32_rn(
                    fmaf(Pi, __uint_as_float(w[e] << 16), -__uint_as_float(r[c * 8 + 2 * e])));
                r[c * 8 + 2 * e + 1] = to_tf32_rn(
                    fmaf(Pi, __uint_as_float(w[e] & 0xffff0000u), -__uint_as_float(r[c * 8 + 2 * e + 1])));
              }
            }
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) r[e] = to_tf32_rn(-__uint_as_float(r[e]));
          }
          tmem_st32(tmem + lane_addr + kColQf + hc * 64 + half * 32, r);
        }
        tmem_wait_st();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar(QF_READY));
        mbar_arrive(bar(QK_FREE));
      }
      item_prev = item;
      if (warp == 4) TCD_STAMP(it, 24);
    }
    if (ok && it > 0) final_epilogue(it - 1, item_prev);
    if (warp == 2 && lane == 0) tma_store_wait_all();
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

#ifdef TV_TC_PROFILE
extern "C" __attribute__((visibility("default"))) int tv_debug_set_tcd_profile(long long* dev_buf) {
  return cudaMemcpyToSymbol(g_tcd_prof, &dev_buf, sizeof(dev_buf)) == cudaSuccess ? 0 : -4;
}
#endif

bool tv_verify_tc_delta_supports(const VerifyArgs& a) {
  return a.bf16 && a.dk == 128 && a.dv == 128 && a.rule == TV_GATED_DELTA && a.T <= kRows &&
         a.tree.max_depth_all < kSlots;
}

int tv_launch_verify_tc_delta(const VerifyArgs& a, int32_t* status, cudaStream_t stream) {
  if (!tv_verify_tc_delta_supports(a)) return TV_ERR_UNSUPPORTED;
  const uint64_t items = (uint64_t)a.L * a.B * a.H;
  const void* const ptrs[5] = {a.q, a.k, a.v, a.S_pre, a.O};
  const MapSet* ms = cached_maps(ptrs, items, a.T, 1, [&](CUtensorMap* m) {
    return make_map(&m[0], a.q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, items, a.T, 128, 64, 64) &&
           make_map(&m[1], a.k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, items, a.T, 128, 64, 64) &&
           make_map(&m[2], a.v, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, items, a.T, 128, 64, 64) &&
           make_map(&m[3], a.S_pre, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, items, 128, 128, 32, 128) &&
           make_map(&m[4], a.O, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, items, a.T, 128, 32, 64);
  });
  if (!ms) return TV_ERR_CUDA;
  static thread_local int configured_dev = -1;
  static thread_local int sm_count = 0;
  int dev = 0;
  TV_CUDA_TRY(cudaGetDevice(&dev));
  if (configured_dev != dev) {
    TV_CUDA_TRY(cudaFuncSetAttribute(verify_tc_delta_kernel,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
    TV_CUDA_TRY(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev));
    configured_dev = dev;
  }
  DeltaParams p;
  p.tree = a.tree;
  p.n_items = (int32_t)items;
  p.B = a.B; p.H = a.H; p.T = a.T;
  p.alpha = a.alpha;
  p.beta = a.beta;
  p.U = a.U;
  p.status = status;
  const int grid = (int)(items < (uint64_t)sm_count ? items : (uint64_t)sm_count);
  verify_tc_delta_kernel<<<grid, kThreads, kSmemBytes, stream>>>(ms->map[0], ms->map[1], ms->map[2], ms->map[3],
                                                                ms->map[4], p);
  TV_CUDA_TRY(cudaGetLastError());
  return TV_OK;
}
