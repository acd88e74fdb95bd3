// Tree verification on the 5th-generation tensor cores (tcgen05 + TMEM + TMA).
//
// Shapes: bf16 q/k/v, fp32 state, dk = dv = 128, T <= 128, gated rule.
// One persistent CTA per SM walks (layer, request, head) items.  Per item
// (Theorem 1 / Eq. 4 with U = V):
//
//   scores  Sc = Q K^T                 bf16 x bf16 -> fp32 in TMEM (exact products)
//   prefix  acc = (2^e_i q_i) S_pre^T  tf32: q widened bf16 -> fp32 and scaled by
//                                      a power of two (exact) into TMEM as the A
//                                      operand; S_pre consumed as raw fp32
//                                      straight from the TMA buffer
//   C'_ij   = 1[j in Anc(i)+{i}] exp2(e_i - g_j) Sc_ij,  g = sum log2(alpha)
//             over the path, e_i = round(g_i) (decay ratios only ever taken on
//             ancestor pairs), split into bf16 hi + lo (~16 mantissa bits)
//   readout acc += C'_hi V + C'_lo V   bf16 x bf16 -> fp32, same accumulator
//   O_i     = exp2(g_i - e_i) acc_i    fp32 epilogue
// The accumulator is double-buffered in TMEM: the epilogue of item n runs under
// the MMAs of item n+1.
//
// S_pre (the HBM-dominant stream) goes TMA -> shared memory -> tensor core and
// is never touched by a thread.  Nothing but O is written.
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer (owns TMEM), warps
// 2..9 = 8 compute warps; compute warp w reads TMEM lanes 32 (w % 4) .. +31
// (the hardware's lane window of that warp) and half of the columns.
// Every wait is an mbarrier wait with a time limit; on expiry the CTA sets the
// status word, drains its own copies and leaves (TMEM is freed on every path).
#include "tv_tc_common.cuh"

namespace {

using namespace tvtc;

constexpr int kThreads = 352;     // producer, MMA issuer, 8 compute warps, output-store warp
constexpr int kComputeWarps = 8;

// shared memory map (byte offsets from the 1024-aligned base)
constexpr uint32_t kOffQ = 0;                     // 2 tiles: k halves of Q  [128][64] bf16
constexpr uint32_t kOffK = kOffQ + 2 * kTile;     // 2 tiles: k halves of K
constexpr uint32_t kOffV = kOffK + 2 * kTile;     // 2 tiles: dv halves of V [128 j][64] bf16
constexpr uint32_t kOffS = kOffV + 2 * kTile;     // 4 tiles: k chunks of S_pre [128 v][32] f32
constexpr uint32_t kOffChi = kOffS + 4 * kTile;   // 2 tiles: j halves of C_hi [128 i][64] bf16
constexpr uint32_t kOffClo = kOffChi + 2 * kTile; // 2 tiles: j halves of C_lo
constexpr uint32_t kOffG = kOffClo + 2 * kTile;   // float g[128]
constexpr uint32_t kOffAl = kOffG + 512;          // float log2(alpha)[128]
constexpr uint32_t kOffF = kOffAl + 512;          // float exp2(-g)[128]
constexpr uint32_t kOffBar = kOffF + 512;         // mbarriers
constexpr uint32_t kOffMisc = kOffBar + 8 * 24;   // tmem base, abort flag
constexpr uint32_t kSmemBytes = kOffMisc + 48 + 1024;  // + alignment slack

enum Bar {
  QK_FULL = 0, QK_FREE, S_FULL, S_FREE, V_FULL, V_FREE,
  SC_DONE, SC_FREE, QF_READY, C_READY, ACC_DONE0, ACC_DONE1, ACC_FREE0, ACC_FREE1, SETUP,
  OST_READY, OST_FREE
};

// TMEM columns: scaled Q (A operand), scores, two output accumulators
constexpr uint32_t kColQf = 0, kColSc = 128, kColAcc0 = 256, kColAcc1 = 384;

constexpr uint32_t kIdescBf16KK = idesc_bf16(128, false);
constexpr uint32_t kIdescBf16KMn = idesc_bf16(128, true);
constexpr uint32_t kIdescTf32 = idesc_tf32(128);

// Eight fp32 values -> bf16 hi and lo parts (hi = upper 16 bits, lo = the exact remainder cut to
// its upper 16 bits: hi + lo carries 16 mantissa bits), stored as two 16-byte chunks.
__device__ __forceinline__ void store_split8(unsigned char* chi, unsigned char* clo, uint32_t off,
                                             const float* cv) {
  uint32_t hi[4], lo[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const uint32_t x0 = __float_as_uint(cv[2 * e]), x1 = __float_as_uint(cv[2 * e + 1]);
    const uint32_t h0 = x0 & 0xffff0000u, h1 = x1 & 0xffff0000u;
    const uint32_t l0 = __float_as_uint(cv[2 * e] - __uint_as_float(h0));
    const uint32_t l1 = __float_as_uint(cv[2 * e + 1] - __uint_as_float(h1));
    hi[e] = __byte_perm(x0, x1, 0x7632);   // {x0.hi16, x1.hi16}
    lo[e] = __byte_perm(l0, l1, 0x7632);
  }
  *reinterpret_cast<uint4*>(chi + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
  *reinterpret_cast<uint4*>(clo + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
}

struct TcParams {
  TreeDev tree;
  int32_t n_items, B, H, T;
  int32_t Hk;  // q/k heads (grouped key heads); H when not grouped
  const float* alpha;
  float* O;
  int32_t* status;
  // packed forest only: request b owns rows offsets[b] .. offsets[b+1]-1 of every plane of
  // `capacity` rows; T is then the per-request node limit (width of the metadata slabs)
  const int32_t* offsets;
  int32_t capacity;
};

__device__ __forceinline__ PackedItem packed_item(const TcParams& p, int item) {
  return tvtc::packed_item(p.offsets, p.B, p.H, p.Hk, item);
}

// PACKED = packed forest: q/k/v/O are planes of `capacity` rows and an item's rows start at its
// request's offset.  Loads take the fixed box at that offset (rows past the request belong to
// other requests and are masked like padding); stores are cut to the request's node count:
// 8-row-aligned part by TMA boxes of 64/32/16/8 rows (tmO, tmO32, tmO16, tmO8), the last < 8
// rows straight from registers.  The dense instantiation ignores the three extra maps.
template <bool PACKED>
__global__ void __launch_bounds__(kThreads, 1)
verify_tc_gated_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmS,
                       const __grid_constant__ CUtensorMap tmO, const __grid_constant__ CUtensorMap tmO32,
                       const __grid_constant__ CUtensorMap tmO16, const __grid_constant__ CUtensorMap tmO8,
                       const TcParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(sm);
  float* g_s = reinterpret_cast<float*>(sm + kOffG);
  float* la_s = reinterpret_cast<float*>(sm + kOffAl);
  float* f_s = reinterpret_cast<float*>(sm + kOffF);
  volatile int* range_ok_s = reinterpret_cast<volatile int*>(sm + kOffMisc + 16);   // [8] per compute warp
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + kOffMisc + 4);
  auto bar = [&](int i) { return sbase + kOffBar + 8u * i; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int T = p.T;
  const int n_jh = T > 64 ? 2 : 1;  // 64-wide j halves that hold real nodes

  if (tid == 0) {
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    mbar_init(bar(QK_FULL), 1);  mbar_init(bar(QK_FREE), 1 + kComputeWarps);
    mbar_init(bar(S_FULL), 1);   mbar_init(bar(S_FREE), 1);
    mbar_init(bar(V_FULL), 1);   mbar_init(bar(V_FREE), 1);
    mbar_init(bar(SC_DONE), 1);  mbar_init(bar(SC_FREE), kComputeWarps);
    mbar_init(bar(QF_READY), kComputeWarps);
    mbar_init(bar(C_READY), kComputeWarps);
    mbar_init(bar(ACC_DONE0), 1); mbar_init(bar(ACC_DONE1), 1);
    mbar_init(bar(ACC_FREE0), kComputeWarps); mbar_init(bar(ACC_FREE1), kComputeWarps);
    mbar_init(bar(SETUP), kComputeWarps);
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
      grid_dependency_wait();   // inputs may come from the kernel in front (dependent launch)
      for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++it) {
        const uint32_t ph = it & 1;
        if (!mbar_wait(bar(QK_FREE), ph ^ 1, abort_flag)) break;
        // packed forest: boxes of 64 rows (per-request limit <= 64) or 128 rows at the request's offset
        const uint32_t box_bytes = PACKED ? (T <= 64 ? kTile / 2 : kTile) : kTile;
        int qk = 0, vplane = item, y0 = 0;
        if constexpr (PACKED) {
          const PackedItem pi = packed_item(p, item);
          qk = pi.plane_qk; vplane = pi.plane_v; y0 = pi.row0;
        } else {
          qk = tv_qk_item(item, p.H, p.Hk);
        }
        mbar_expect_tx(bar(QK_FULL), 4 * box_bytes);
        tma_load_3d(sbase + kOffQ, &tmQ, bar(QK_FULL), 0, y0, qk);
        tma_load_3d(sbase + kOffQ + kTile, &tmQ, bar(QK_FULL), 64, y0, qk);
        tma_load_3d(sbase + kOffK, &tmK, bar(QK_FULL), 0, y0, qk);
        tma_load_3d(sbase + kOffK + kTile, &tmK, bar(QK_FULL), 64, y0, qk);
        pend_qk = 1 + (int)ph;
        if (!mbar_wait(bar(S_FREE), ph ^ 1, abort_flag)) break;
        mbar_expect_tx(bar(S_FULL), 4 * kTile);
#pragma unroll
        for (int c = 0; c < 4; ++c)
          tma_load_3d(sbase + kOffS + c * kTile, &tmS, bar(S_FULL), 32 * c, 0, item);
        pend_s = 1 + (int)ph;
        if (!mbar_wait(bar(V_FREE), ph ^ 1, abort_flag)) break;
        mbar_expect_tx(bar(V_FULL), 2 * box_bytes);
        tma_load_3d(sbase + kOffV, &tmV, bar(V_FULL), 0, y0, vplane);
        tma_load_3d(sbase + kOffV + kTile, &tmV, bar(V_FULL), 64, y0, vplane);
        pend_v = 1 + (int)ph;
      }
      if (*abort_flag) {
        // Leave no copy of ours in flight: wait (bounded) for the last loads issued.
        if (pend_qk) mbar_wait(bar(QK_FULL), pend_qk - 1, abort_flag + 1);
        if (pend_s) mbar_wait(bar(S_FULL), pend_s - 1, abort_flag + 1);
        if (pend_v) mbar_wait(bar(V_FULL), pend_v - 1, abort_flag + 1);
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    if (lane == 0) {
      uint32_t it = 0;
      for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++it) {
        const uint32_t ph = it & 1;
        const uint32_t acc_col = (it & 1) ? kColAcc1 : kColAcc0;
        const int acc_done = (it & 1) ? ACC_DONE1 : ACC_DONE0;
        const int acc_free = (it & 1) ? ACC_FREE1 : ACC_FREE0;
        const uint32_t ph2 = (it >> 1) & 1;   // the two accumulators alternate
        // scores = Q K^T
        if (!mbar_wait(bar(QK_FULL), ph, abort_flag)) break;
        if (!mbar_wait(bar(SC_FREE), ph ^ 1, abort_flag)) break;
        tc_fence_after();
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int s = 0; s < 4; ++s)
            mma_bf16_ss(tmem + kColSc, desc_kmajor(sbase + kOffQ + h * kTile + s * 32),
                        desc_kmajor(sbase + kOffK + h * kTile + s * 32), kIdescBf16KK, (h | s) != 0);
        tc_commit(bar(SC_DONE));
        tc_commit(bar(QK_FREE));
        // acc = (2^e Q) S_pre^T  (A = scaled Q as fp32 in TMEM, B = S_pre chunks)
        if (!mbar_wait(bar(S_FULL), ph, abort_flag)) break;
        if (!mbar_wait(bar(QF_READY), ph, abort_flag)) break;
        if (!mbar_wait(bar(acc_free), ph2 ^ 1, abort_flag)) break;
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int s = 0; s < 4; ++s)
            mma_tf32_ts(tmem + acc_col, tmem + kColQf + c * 32 + s * 8,
                        desc_kmajor(sbase + kOffS + c * kTile + s * 32), kIdescTf32, (c | s) != 0);
        tc_commit(bar(S_FREE));
        // acc += C'_hi V + C'_lo V
        if (!mbar_wait(bar(C_READY), ph, abort_flag)) break;
        if (!mbar_wait(bar(V_FULL), ph, abort_flag)) break;
        tc_fence_after();
        for (int jh = 0; jh < n_jh; ++jh)
#pragma unroll
          for (int s = 0; s < 4; ++s) {
            const uint64_t bdesc = desc_mnmajor(sbase + kOffV + (jh * 4 + s) * 2048, kTile);
            mma_bf16_ss(tmem + acc_col, desc_kmajor(sbase + kOffChi + jh * kTile + s * 32), bdesc,
                        kIdescBf16KMn, 1);
            mma_bf16_ss(tmem + acc_col, desc_kmajor(sbase + kOffClo + jh * kTile + s * 32), bdesc,
                        kIdescBf16KMn, 1);
          }
        tc_commit(bar(V_FREE));
        tc_commit(bar(acc_done));
      }
    }
  } else if (warp == kComputeWarps + 2) {
    // ===================== output stores =====================
    // The staged chunks of an item leave by TMA once all compute warps have written them
    // (OST_READY); OST_FREE tells them that the chunks have been read.  T <= 64: the chunks are
    // not the C' tiles, and OST_FREE phase k says that the store of item k-1 is read (phase 0
    // is given away up front).  T > 64: phase k = the store of item k.
    if (lane == 0) {
      const bool small = T <= 64;
      auto stage_addr = [&](int c4) -> uint32_t {
        return small ? kOffChi + kTile + (uint32_t)(c4 >> 1) * (kOffClo - kOffChi) + (uint32_t)(c4 & 1) * 8192u
                     : kOffChi + (uint32_t)c4 * kTile;
      };
      if (small) mbar_arrive(bar(OST_FREE));
      uint32_t it = 0;
      for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++it) {
        if (!mbar_wait(bar(OST_READY), it & 1, abort_flag)) break;
        if constexpr (PACKED) {
          // groups of 8 rows, largest boxes first; staging rows r.. start on a 1024-byte
          // boundary, so the swizzle phase of a partial box equals that of the full tile
          const PackedItem pk = packed_item(p, item);
          const int full = pk.n & ~7;
          int r = 0;
          auto put = [&](const CUtensorMap* m, int rows_box) {
            while (full - r >= rows_box) {
#pragma unroll
              for (int c = 0; c < 4; ++c)
                tma_store_3d(m, sbase + stage_addr(c) + (uint32_t)r * 128u, 32 * c, pk.row0 + r, pk.plane_v);
              r += rows_box;
            }
          };
          put(&tmO, 64);
          put(&tmO32, 32);
          put(&tmO16, 16);
          put(&tmO8, 8);
        } else {
#pragma unroll
          for (int c = 0; c < 4; ++c) tma_store_3d(&tmO, sbase + stage_addr(c), 32 * c, 0, item);
        }
        tma_store_commit();
        tma_store_wait_read();
        mbar_arrive(bar(OST_FREE));
      }
      tma_store_wait_all();   // our stores are complete before we leave
    }
  } else {
    // ===================== compute warps =====================
    const int cw = warp - 2;
    const int quad = warp & 3;          // TMEM lane window of this warp
    const int hc = cw >> 2;             // column half handled by this warp
    const int row = quad * 32 + lane;   // node i
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t swz = (uint32_t)(row & 7);
    const bool warp_live = quad * 32 < T;   // this warp's 32 rows hold at least one node

    // O_i = r_i acc_i for the item whose accumulator is `it_prev`: TMEM -> registers -> the
    // (now idle) C' tiles as four [128 rows][32 fp32] swizzled tiles -> one TMA store per tile
    // (full 128-byte lines; rows past T are clipped by the tensor map).
    // T <= 64: the j >= 64 halves of the C' tiles are idle and hold the staging chunks
    // ([64 rows][32 fp32], 8 KiB each), so staging never collides with the C' tiles of the
    // next item and the store is only waited for one item later.  T > 64: the chunks are the
    // four C' tiles themselves and the store must have read them before C' is rewritten.
    const bool small = T <= 64;
    auto stage_addr = [&](int c4) -> uint32_t {
      return small ? kOffChi + kTile + (uint32_t)(c4 >> 1) * (kOffClo - kOffChi) + (uint32_t)(c4 & 1) * 8192u
                   : kOffChi + (uint32_t)c4 * kTile;
    };
    auto final_epilogue = [&](uint32_t it_prev, int item_prev, float r_prev, uint32_t ost_phase,
                              const PackedItem& pk_prev) -> bool {
      const int acc_done = (it_prev & 1) ? ACC_DONE1 : ACC_DONE0;
      const int acc_free = (it_prev & 1) ? ACC_FREE1 : ACC_FREE0;
      const uint32_t acc_col = (it_prev & 1) ? kColAcc1 : kColAcc0;
      // T <= 64: the store of the item before has read the staging chunks
      if (small && !mbar_wait_warp(bar(OST_FREE), ost_phase, abort_flag)) return false;
      if (!mbar_wait_warp(bar(acc_done), (it_prev >> 1) & 1, abort_flag)) return false;
      tc_fence_after();
      if (warp_live) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t r1[32];
          tmem_ld32(tmem + lane_addr + acc_col + hc * 64 + half * 32, r1);
          tmem_wait_ld();
          unsigned char* orow = sm + stage_addr(hc * 2 + half) + row * 128;
          // packed forest: the rows after the last full group of 8 leave from registers
          const bool tail_row = PACKED && row >= (pk_prev.n & ~7) && row < pk_prev.n;
          float* otail = nullptr;
          if constexpr (PACKED)
            otail = p.O + ((size_t)pk_prev.plane_v * p.capacity + pk_prev.row0 + row) * 128 + hc * 64 + half * 32;
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            float4 o;
            o.x = r_prev * __uint_as_float(r1[4 * c + 0]);
            o.y = r_prev * __uint_as_float(r1[4 * c + 1]);
            o.z = r_prev * __uint_as_float(r1[4 * c + 2]);
            o.w = r_prev * __uint_as_float(r1[4 * c + 3]);
            *reinterpret_cast<float4*>(orow + (((uint32_t)c ^ swz) << 4)) = o;
            if (tail_row) *reinterpret_cast<float4*>(otail + 4 * c) = o;
          }
        }
      }
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar(acc_free));
        mbar_arrive(bar(OST_READY));
      }
      return small ? true : mbar_wait_warp(bar(OST_FREE), ost_phase, abort_flag);
    };

    // metadata of the first item; later items are fetched one item ahead
    uint64_t nm0 = 0, nm1 = 0;
    float nal = 1.f;   // raw decay gate of the next item (log2 taken when it is used)
    PackedItem npk = {0, 0, 0, 0, T};   // packed forest: rows of the next item
    auto fetch_meta = [&](int item) {
      nm0 = 0; nm1 = 0; nal = 1.f;
      if constexpr (PACKED) {
        if (item < p.n_items) {
          npk = packed_item(p, item);
          if (row < npk.n) {
            const uint64_t* m = p.tree.anc + ((size_t)npk.b * T + row) * 2;
            nm0 = m[0];
            nm1 = m[1];
            nal = p.alpha[(size_t)npk.plane_v * p.capacity + npk.row0 + row];
          }
        }
      } else if (item < p.n_items && row < T) {
        const int b = (item / p.H) % p.B;
        const int tb = p.tree.n_trees == 1 ? 0 : b;
        const uint64_t* m = p.tree.anc + ((size_t)tb * T + row) * 2;
        nm0 = m[0];
        nm1 = m[1];
        nal = p.alpha[(size_t)item * T + row];
      }
    };
    // dependent launch: barrier set-up and the TMEM allocation above ran under the tail of the
    // kernel in front; everything that reads global memory waits for it here
    grid_dependency_wait();
    // the commit kernel behind this one may be scheduled as SMs drain (it orders itself)
    if (warp == 2 && lane == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    fetch_meta(blockIdx.x);

    uint32_t it = 0;
    bool ok = true;
    int item_prev = 0;
    float r_prev = 0.f;
    PackedItem pk = npk, pk_prev = npk;
    const int total_rows = PACKED ? p.offsets[p.B] : 0;   // rows at and past this one hold no node
    for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++it) {
      const uint32_t ph = it & 1;
      uint64_t m0 = nm0, m1 = nm1;
      pk = npk;
      const int Tb = PACKED ? pk.n : T;   // real nodes of this item
      // ---- path decay: g_i = sum of log2(alpha) over Anc(i) + {i} ----
      const float la_own = log2f(nal);
      if (hc == 0 && row < Tb) la_s[row] = la_own;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(SETUP));
      fetch_meta(item + (int)gridDim.x);   // next item's metadata rides under this item's work
      if (!(ok = mbar_wait_warp(bar(SETUP), 0, abort_flag))) break;   // SETUP: two phases per item
      float g = 0.f;
      if (row < Tb) {
        g = la_own;
        uint64_t a0 = m0, a1 = m1;
        while (a0) { const int j = __ffsll((long long)a0) - 1; a0 &= a0 - 1; g += la_s[j]; }
        while (a1) { const int j = __ffsll((long long)a1) - 1; a1 &= a1 - 1; g += la_s[64 + j]; }
        if (row < 64) m0 |= 1ull << row; else m1 |= 1ull << (row - 64);   // M+ = M- + I
      }
      if (hc == 0 && row < Tb) {
        g_s[row] = g;
        f_s[row] = exp2f(-g);
      }
      // exp2(e_i - g_j) = 2^e_i * 2^-g_j is safe when every |g| <= 100; otherwise take exp2 per pair
      const bool range_ok_warp = __all_sync(0xffffffffu, row >= Tb || fabsf(g) <= 100.f);
      if (lane == 0) range_ok_s[cw] = range_ok_warp;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(SETUP));
      // Row scaling.  The accumulator holds  2^e (q_i S_pre^T) + sum_j 2^(e - g_j) s_ij v_j  and
      // O_i = 2^(g_i - e) acc: e is an integer, so the scaled q stays exact in tf32, and the
      // exponents e - g_j = (e - g_i) + (g_i - g_j) stay small on ancestor pairs.  Below 2^-100
      // the prefix term is under fp32 resolution of anything it is added to and is dropped.
      const bool tiny = g < -100.f;
      const float e_int = tiny ? g : fminf(rintf(g), 100.f);
      const float a_scale = tiny ? 0.f : exp2f(e_int);
      const float r_scale = exp2f(g - e_int);
      // ---- Q row (bf16, swizzled tile) -> scaled fp32 -> TMEM (A operand of the prefix MMA) ----
      if (!(ok = mbar_wait_warp(bar(QK_FULL), ph, abort_flag))) break;
      if (!(ok = mbar_wait_warp(bar(S_FREE), ph ^ 1, abort_flag))) break;   // prefix MMA of item-1 done with Qf
      tc_fence_after();
      if (warp_live) {
        const unsigned char* qrow = sm + kOffQ + hc * kTile + row * 128;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t r[32];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const uint4 x = *reinterpret_cast<const uint4*>(qrow + (((half * 4 + c) ^ swz) << 4));
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              r[c * 8 + 2 * e] = __float_as_uint(a_scale * __uint_as_float(w[e] << 16));
              r[c * 8 + 2 * e + 1] = __float_as_uint(a_scale * __uint_as_float(w[e] & 0xffff0000u));
            }
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
      // ---- scores -> masked, decayed, split C' ----
      if (!(ok = mbar_wait_warp(bar(SC_DONE), ph, abort_flag))) break;
      if (!(ok = mbar_wait_warp(bar(SETUP), 1, abort_flag))) break;
      // ---- output rows of the previous item: its accumulator is complete once its readout MMA
      // is, and the C' tiles it frees double as the staging area of the output store ----
      if (it > 0 && !(ok = final_epilogue(it - 1, item_prev, r_prev, (it - 1) & 1, pk_prev))) break;
      tc_fence_after();
      if (warp_live) {
        bool fast = true;
#pragma unroll
        for (int w8 = 0; w8 < kComputeWarps; ++w8) fast = fast && range_ok_s[w8];
        // this warp covers 32 n_jh of the 64 n_jh real columns, 32 at a time
        for (int h = 0; h < n_jh; ++h) {
          const int cbase = hc * 32 * n_jh + h * 32;     // first column j of this group
          uint32_t r[32];
          tmem_ld32(tmem + lane_addr + kColSc + cbase, r);
          tmem_wait_ld();
          const uint32_t bits = cbase < 64 ? (uint32_t)(m0 >> cbase) : (uint32_t)(m1 >> (cbase - 64));
          unsigned char* chi = sm + kOffChi + (cbase >> 6) * kTile + row * 128;
          unsigned char* clo = sm + kOffClo + (cbase >> 6) * kTile + row * 128;
          const int chunk0 = (cbase & 63) >> 3;
          if (fast) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const float4 fa = *reinterpret_cast<const float4*>(f_s + cbase + c * 8);
              const float4 fb = *reinterpret_cast<const float4*>(f_s + cbase + c * 8 + 4);
              const float f8[8] = {fa.x, fa.y, fa.z, fa.w, fb.x, fb.y, fb.z, fb.w};
              float cv[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const float x = __uint_as_float(r[c * 8 + e]) * (a_scale * f8[e]);
                cv[e] = ((bits >> (c * 8 + e)) & 1u) ? x : 0.f;   // select, never 0 * x
              }
              store_split8(chi, clo, ((uint32_t)((chunk0 + c) ^ swz)) << 4, cv);
            }
          } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              float cv[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const float x = __uint_as_float(r[c * 8 + e]) * exp2f(e_int - g_s[cbase + c * 8 + e]);
                cv[e] = ((bits >> (c * 8 + e)) & 1u) ? x : 0.f;
              }
              store_split8(chi, clo, ((uint32_t)((chunk0 + c) ^ swz)) << 4, cv);
            }
          }
        }
      }
      if constexpr (PACKED) {
        // A box that reaches past the last node of the forest brings rows nobody wrote: zero them
        // in the V tiles (0 x garbage would not be 0); K and Q rows are masked by selection.
        const int box_rows = T <= 64 ? 64 : 128;
        if (pk.row0 + box_rows > total_rows) {
          if (!(ok = mbar_wait_warp(bar(V_FULL), ph, abort_flag))) break;
          if (row >= total_rows - pk.row0 && row < box_rows) {
            uint4* vrow = reinterpret_cast<uint4*>(sm + kOffV + hc * kTile + row * 128);
#pragma unroll
            for (int c = 0; c < 8; ++c) vrow[c] = make_uint4(0u, 0u, 0u, 0u);
          }
        }
      }
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar(C_READY));
        mbar_arrive(bar(SC_FREE));
      }
      item_prev = item;
      r_prev = r_scale;
      pk_prev = pk;
    }
    if (ok && it > 0) final_epilogue(it - 1, item_prev, r_prev, (it - 1) & 1, pk_prev);
  }

  // ---- teardown: every path comes here ----
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u)
                 : "memory");
  }
  if (tid == 0 && *abort_flag && p.status) atomicExch(p.status, (int)TV_ERR_DEVICE_TIMEOUT);
}

// ---------------------------------------------------------------------------
// Host side: tensor maps and launch.
// ---------------------------------------------------------------------------
// Gated rule: the correction rows are the values themselves (U = V).
__global__ void widen_bf16_kernel(const __nv_bfloat16* __restrict__ v, float* __restrict__ U, size_t n8) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n8; i += (size_t)gridDim.x * blockDim.x) {
    const uint4 x = reinterpret_cast<const uint4*>(v)[i];
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
    float4 a, b;
    a.x = __uint_as_float(w[0] << 16); a.y = __uint_as_float(w[0] & 0xffff0000u);
    a.z = __uint_as_float(w[1] << 16); a.w = __uint_as_float(w[1] & 0xffff0000u);
    b.x = __uint_as_float(w[2] << 16); b.y = __uint_as_float(w[2] & 0xffff0000u);
    b.z = __uint_as_float(w[3] << 16); b.w = __uint_as_float(w[3] & 0xffff0000u);
    reinterpret_cast<float4*>(U)[2 * i] = a;
    reinterpret_cast<float4*>(U)[2 * i + 1] = b;
  }
}

// Packed forest: only the rows that hold nodes, plane by plane.
__global__ void widen_bf16_rows_kernel(const __nv_bfloat16* __restrict__ v, float* __restrict__ U, size_t planes,
                                       size_t capacity, const int32_t* __restrict__ offsets, int n_req) {
  const size_t n8 = (size_t)offsets[n_req] * 128 / 8;   // 16-byte groups of one plane that hold nodes
  for (size_t pl = blockIdx.y; pl < planes; pl += gridDim.y) {
    const uint4* src = reinterpret_cast<const uint4*>(v + pl * capacity * 128);
    float4* dst = reinterpret_cast<float4*>(U + pl * capacity * 128);
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n8; i += (size_t)gridDim.x * blockDim.x) {
      const uint4 x = src[i];
      const uint32_t w[4] = {x.x, x.y, x.z, x.w};
      float4 a, b;
      a.x = __uint_as_float(w[0] << 16); a.y = __uint_as_float(w[0] & 0xffff0000u);
      a.z = __uint_as_float(w[1] << 16); a.w = __uint_as_float(w[1] & 0xffff0000u);
      b.x = __uint_as_float(w[2] << 16); b.y = __uint_as_float(w[2] & 0xffff0000u);
      b.z = __uint_as_float(w[3] << 16); b.w = __uint_as_float(w[3] & 0xffff0000u);
      dst[2 * i] = a;
      dst[2 * i + 1] = b;
    }
  }
}

}  // namespace

// Self-test of the bounded wait every tensor-core kernel relies on: one CTA waits, with a short
// limit, on a barrier that nothing ever arrives at, then reports and returns like the kernels do.
namespace {
__global__ void wait_timeout_selftest_kernel(int32_t* status) {
  __shared__ uint64_t bar_mem;
  __shared__ int abort_flag;
  const uint32_t bar = smem_u32(&bar_mem);
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const bool ok = mbar_wait_warp(bar, 0, &abort_flag, 1ll << 22);   // ~2 ms, never satisfied
  __syncthreads();
  if (threadIdx.x == 0) atomicExch(status, ok ? (int)TV_OK : (int)TV_ERR_DEVICE_TIMEOUT);
}
}  // namespace

extern "C" __attribute__((visibility("default"))) int tv_selftest_wait_timeout(int32_t* status, void* stream) {
  if (!status || ((uintptr_t)status & 3)) return TV_ERR_BAD_ARG;
  wait_timeout_selftest_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(status);
  TV_CUDA_TRY(cudaGetLastError());
  return TV_OK;
}

bool tv_verify_tc_supports(const VerifyArgs& a) {
  return a.bf16 && a.dk == 128 && a.dv == 128 && a.rule == TV_GATED && a.T <= 128;
}

int tv_launch_verify_tc(const VerifyArgs& a, int32_t* status, cudaStream_t stream) {
  if (!tv_verify_tc_supports(a)) return TV_ERR_UNSUPPORTED;
  const bool packed = a.tree.offsets != nullptr;
  const uint64_t items = (uint64_t)a.L * a.B * a.H;
  const uint64_t qk_items = (uint64_t)a.L * a.B * a.Hk;
  const uint32_t orows = a.T <= 64 ? 64 : 128;   // rows of one staged output chunk
  const void* const ptrs[5] = {a.q, a.k, a.v, a.S_pre, a.O};
  const MapSet* ms = nullptr;
  const MapSet* mo = nullptr;   // packed forest: output boxes of 32, 16 and 8 rows
  if (!packed) {
    ms = cached_maps(ptrs, items, a.T, a.Hk << 8, [&](CUtensorMap* m) {
      return make_map(&m[0], a.q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, qk_items, a.T, 128, 64) &&
             make_map(&m[1], a.k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, qk_items, a.T, 128, 64) &&
             make_map(&m[2], a.v, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, items, a.T, 128, 64) &&
             make_map(&m[3], a.S_pre, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, items, 128, 128, 32) &&
             make_map(&m[4], a.O, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, items, a.T, 128, 32, orows);
    });
    mo = ms;
  } else {
    // planes of `capacity` rows; loads in boxes of 64 or 128 rows, stores in boxes of 64/32/16/8
    const uint64_t cap = (uint64_t)a.tree.capacity;
    const uint64_t pv = (uint64_t)a.L * a.H, pqk = (uint64_t)a.L * a.Hk;
    const uint32_t lrows = a.T <= 64 ? 64 : 128;
    const uint64_t key = (cap << 24) ^ items;
    ms = cached_maps(ptrs, key, a.T, 4 | (a.Hk << 8), [&](CUtensorMap* m) {
      return make_map(&m[0], a.q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, pqk, cap, 128, 64, lrows) &&
             make_map(&m[1], a.k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, pqk, cap, 128, 64, lrows) &&
             make_map(&m[2], a.v, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, pv, cap, 128, 64, lrows) &&
             make_map(&m[3], a.S_pre, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, items, 128, 128, 32) &&
             make_map(&m[4], a.O, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, pv, cap, 128, 32, 64);
    });
    const void* const optrs[5] = {a.O, nullptr, nullptr, nullptr, nullptr};
    mo = cached_maps(optrs, key, a.T, 5, [&](CUtensorMap* m) {
      return make_map(&m[0], a.O, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, pv, cap, 128, 32, 32) &&
             make_map(&m[1], a.O, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, pv, cap, 128, 32, 16) &&
             make_map(&m[2], a.O, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, pv, cap, 128, 32, 8);
    });
  }
  if (!ms || !mo) return TV_ERR_CUDA;
  static thread_local int configured_dev = -1;
  static thread_local int sm_count = 0;
  int dev = 0;
  TV_CUDA_TRY(cudaGetDevice(&dev));
  if (configured_dev != dev) {
    TV_CUDA_TRY(cudaFuncSetAttribute(verify_tc_gated_kernel<false>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
    TV_CUDA_TRY(cudaFuncSetAttribute(verify_tc_gated_kernel<true>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
    TV_CUDA_TRY(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev));
    configured_dev = dev;
  }
  TcParams p;
  p.tree = a.tree;
  p.n_items = (int32_t)items;
  p.B = a.B; p.H = a.H; p.T = a.T; p.Hk = a.Hk;
  p.alpha = a.alpha;
  p.O = a.O;
  p.status = status;
  p.offsets = a.tree.offsets;
  p.capacity = a.tree.capacity;
  const int grid = (int)(items < (uint64_t)sm_count ? items : (uint64_t)sm_count);
  if (packed) {
    TV_CUDA_TRY(launch_dependent(verify_tc_gated_kernel<true>, grid, kThreads, kSmemBytes, stream, ms->map[0],
                                 ms->map[1], ms->map[2], ms->map[3], ms->map[4], mo->map[0], mo->map[1],
                                 mo->map[2], p));
    if (a.U) {
      const size_t planes = (size_t)a.L * a.H;
      widen_bf16_rows_kernel<<<dim3(64, (unsigned)(planes < 65535 ? planes : 65535)), 256, 0, stream>>>(
          reinterpret_cast<const __nv_bfloat16*>(a.v), a.U, planes, (size_t)a.tree.capacity, a.tree.offsets, a.B);
      TV_CUDA_TRY(cudaGetLastError());
    }
    return TV_OK;
  }
  TV_CUDA_TRY(launch_dependent(verify_tc_gated_kernel<false>, grid, kThreads, kSmemBytes, stream, ms->map[0],
                               ms->map[1], ms->map[2], ms->map[3], ms->map[4], ms->map[4], ms->map[4],
                               ms->map[4], p));
  if (a.U) {
    const size_t n8 = items * a.T * 128 / 8;
    const int blocks = (int)((n8 + 255) / 256 < 4096 ? (n8 + 255) / 256 : 4096);
    widen_bf16_kernel<<<blocks, 256, 0, stream>>>(reinterpret_cast<const __nv_bfloat16*>(a.v), a.U, n8);
    TV_CUDA_TRY(cudaGetLastError());
  }
  return TV_OK;
}
