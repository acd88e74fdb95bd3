// Tree verification on the 5th-generation tensor cores (tcgen05 + TMEM + TMA).
//
// Shapes: bf16 q/k/v, fp32 state, dk = dv = 128 (or 64, dense layouts), T <= 128, gated rule.
// The text below is written for 128.
// One persistent CTA per SM walks (layer, request, head) items.  Per item
// (Theorem 1 / Eq. 4 with U = V):
//
//   scores  Sc = Q K^T                 bf16 x bf16 -> fp32 in TMEM (exact products)
//   prefix  acc = q_i S_pre^T          bf16 x bf16 -> fp32.  A operand: the q rows, copied to TMEM
//                                      as packed bf16.  B operand: S_pre split into bf16
//                                      hi + lo (16 mantissa bits, both rounded to nearest)
//                                      IN PLACE in the buffer the TMA filled: the fp32 row
//                                      halves k 0..31 | 32..63 of a state row become its hi row
//                                      and its lo row of 64 bf16 -- same bytes, same swizzle.
//   C'_ij   = 1[j in Anc(i)+{i}] 2^(-g_j) Sc_ij,  g = sum log2(alpha) over the path (decay
//             ratios only ever taken on ancestor pairs), split into bf16 hi + lo
//   readout acc += C'_hi V + C'_lo V   bf16 x bf16 -> fp32, same accumulator
//   O_i     = 2^(g_i) acc_i            fp32 epilogue
// The accumulator is double-buffered in TMEM: the epilogue of item n runs under
// the MMAs of item n+1.
//
// Extreme decay.  The plain form above is used as long as every |g| <= 100.  Otherwise a row
// exponent e_i = round(g_i) keeps every factor in range: the compute warps replace the q rows
// in TMEM by 2^e_i q_i (exact in bf16), C'_ij = 2^(e_i - g_j) Sc_ij, O_i = 2^(g_i - e_i) acc;
// rows with g_i < -100 drop the prefix term, which is below fp32 resolution of anything it is
// added to.
//
// Why the state is split rather than fed to the tensor core as fp32 (kind::tf32 cuts the
// mantissa to 10 bits): a state that has absorbed many rank-one updates is dominated by a
// few directions, a query nearly orthogonal to them sums large terms that cancel, and the
// tf32 cut of those terms reached 1e-2 of the output in such states (5e-4 on unstructured
// ones).  The split keeps 16 bits (worst case seen 4e-4, typically 1e-5), costs the
// tensor time of the tf32 product, and needs no extra shared memory.
//
// T <= 64 (SMALL): operand boxes of 64 rows, and the shared memory that frees holds a second
// stage of S_pre, so that the state of item n+1 (the HBM-dominant stream) is in flight while
// item n is worked on.  T > 64: one stage of everything.
//
// Warp roles, in groups of four warps so that registers can be moved between them
// (setmaxnreg).  Whatever depends on loaded data only is taken off the compute warps' chain.
//   warps 0..3   service, 64 registers: 0 = TMA producer (one thread polls the gates of three
//                independent load streams: q+k, v, S_pre), 1 = MMA issuer (owns TMEM), 2 = issues
//                the output stores, 3 = path decay: g, 2^-g and the range flag of item n+1 and
//                n+2 by pointer jumping over the tree, into one of two shared-memory copies
//   warps 4..11  compute, 168 registers: O of item n-1 from the accumulator, then C' of item n
//                from the scores; warp w reads TMEM lanes 32 (w % 4) .. +31 (the hardware's lane
//                window of that warp) and half of the columns
//   warps 12..15 operands, 104 registers, thread r = node r = state row r: the q rows into TMEM
//                (two copies, items alternate), the split of S_pre
// The code is kept small where that is free (one output site, a short bounded wait, division
// by launch constants as multiply-shift): the five roles share one instruction cache, and at
// 79 KB of code it hit in 59 % of its requests.
// Every wait is an mbarrier wait with a time limit; on expiry the CTA sets the status word,
// drains its own copies and leaves (TMEM is freed on every path).
#include "tv_tc_common.cuh"

namespace {

using namespace tvtc;

constexpr int kThreads = 512;     // 4 service warps, 8 compute warps, 4 operand warps
constexpr int kComputeWarps = 8;
constexpr int kFirstComputeWarp = 4;
constexpr int kFirstSplitWarp = 12;
constexpr int kSplitWarps = 4;

// Shared memory map (byte offsets from the 1024-aligned base).  An MMA with M = 128 reads 128
// rows of its A tile whatever T is: with 64-row boxes the rows 64..127 it reads are the bytes
// of the next buffer; they only reach accumulator rows >= 64, which nobody reads.
template <bool SMALL>
struct Lay {
  static constexpr uint32_t kBox = SMALL ? kTile / 2 : kTile;   // one operand box: [64 | 128 rows][64 bf16]
  static constexpr int kStages = SMALL ? 2 : 1;                 // stages of S_pre
  static constexpr uint32_t kOffQ = 0;                          // 2 boxes: k halves of Q
  static constexpr uint32_t kOffK = kOffQ + 2 * kBox;           // 2 boxes: k halves of K
  static constexpr uint32_t kOffV = kOffK + 2 * kBox;           // 2 boxes: dv halves of V [j][64]
  static constexpr uint32_t kOffS = kOffV + 2 * kBox;           // per stage 4 tiles [128 v][128 B]: fp32 k chunks,
                                                                // after the split: hi | lo | hi | lo of the k halves
  static constexpr uint32_t kOffChi = kOffS + kStages * 4 * kTile;   // C'_hi: j halves [128 i][64] (SMALL: one, 64 rows live)
  static constexpr uint32_t kOffClo = kOffChi + (SMALL ? kBox : 2 * kTile);
  // output staging: four chunks [64 | 128 rows][32 fp32].  SMALL: a region of its own; else the
  // four C' tiles themselves, idle once the readout MMAs of the item are complete
  static constexpr uint32_t kOffStage = SMALL ? kOffClo + kBox : kOffChi;
  static constexpr uint32_t kStageChunk = SMALL ? kTile / 2 : kTile;
  // path decay of two items in flight: g[2][kNodes], exp2(-g)[2][kNodes]; log2(alpha)[kNodes] is
  // the decay warp's own scratch
  static constexpr uint32_t kNodes = SMALL ? 64 : 128;
  static constexpr uint32_t kOffG = SMALL ? kOffStage + 4 * kStageChunk : kOffClo + 2 * kTile;
  static constexpr uint32_t kOffF = kOffG + 2 * kNodes * 4;
  static constexpr uint32_t kOffAl = kOffF + 2 * kNodes * 4;
  static constexpr uint32_t kOffBar = kOffAl + kNodes * 4;   // mbarriers
  static constexpr uint32_t kOffMisc = kOffBar + 8 * 32;     // tmem base, abort flags, range flags of two items
  // The dynamic shared memory of a CTA starts on a 1024-byte boundary (asked for in the
  // declaration and checked at entry), so there is no alignment slack in this figure.
  static constexpr uint32_t kSmemBytes = kOffMisc + 32;
  static_assert(kSmemBytes <= 232448, "shared memory of one CTA");
};

enum Bar {
  QK_FULL = 0, QK_FREE, S_FULL0, S_FULL1, S_CONV0, S_CONV1, S_FREE0, S_FREE1, V_FULL, V_FREE,
  SC_DONE, SC_FREE, QB_READY0, QB_READY1, QS_READY0, QS_READY1, C_READY, ACC_DONE0, ACC_DONE1, ACC_FREE0, ACC_FREE1,
  META_READY0, META_READY1, META_FREE0, META_FREE1, OST_READY, OST_FREE, kNumBars
};
static_assert(kNumBars <= 32, "barrier area");

// TMEM columns: Q as packed bf16 (A operand of the prefix MMA; two copies of 64 columns, items
// alternate), scores, two accumulators
constexpr uint32_t kColQb = 0, kColSc = 128, kColAcc0 = 256, kColAcc1 = 384;

constexpr uint32_t kIdescKK128 = idesc_bf16(128, false);
constexpr uint32_t kIdescKK64 = idesc_bf16(64, false);

__device__ __forceinline__ void mma_bf16_ts(uint32_t d, uint32_t a_tmem, uint64_t b, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d), "r"(a_tmem), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}

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

// Two fp32 -> one word of two bf16, rounded to nearest even (first argument in the low half).
__device__ __forceinline__ uint32_t pack_bf16_rn(float lo_elem, float hi_elem) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi_elem), "f"(lo_elem));
  return r;
}

// The state split.  Thread (row v, k half p) owns the two 128-byte rows that hold
// S_pre[v][64 p .. 64 p + 63] as fp32 (row v of tiles 2p and 2p + 1 of the stage, 128-byte
// swizzle) and rewrites them as 64 bf16 hi values (tile 2p) and 64 bf16 lo values (tile 2p + 1)
// in the K-major swizzled layout the MMA reads: hi = rn(x), lo = rn(x - hi), x - hi exact.
// Everything is read before anything is written; no other thread touches these rows.
__device__ __forceinline__ void split_state_row(unsigned char* stage, int row, int p, uint32_t swz) {
  unsigned char* r0 = stage + (uint32_t)(2 * p) * kTile + (uint32_t)row * 128u;
  unsigned char* r1 = r0 + kTile;
  uint4 hi[8], lo[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) {   // output chunk c = k 8c .. 8c + 7 of this half
    const unsigned char* src = c < 4 ? r0 : r1;
    const uint32_t f = (uint32_t)(c & 3) * 2u;
    const float4 a = *reinterpret_cast<const float4*>(src + ((f ^ swz) << 4));
    const float4 b = *reinterpret_cast<const float4*>(src + (((f + 1u) ^ swz) << 4));
    const float x[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint32_t h[4], l[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      h[e] = pack_bf16_rn(x[2 * e], x[2 * e + 1]);
      const float l0 = x[2 * e] - __uint_as_float(h[e] << 16);
      const float l1 = x[2 * e + 1] - __uint_as_float(h[e] & 0xffff0000u);
      l[e] = pack_bf16_rn(l0, l1);
    }
    hi[c] = make_uint4(h[0], h[1], h[2], h[3]);
    lo[c] = make_uint4(l[0], l[1], l[2], l[3]);
  }
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    *reinterpret_cast<uint4*>(r0 + (((uint32_t)c ^ swz) << 4)) = hi[c];
    *reinterpret_cast<uint4*>(r1 + (((uint32_t)c ^ swz) << 4)) = lo[c];
  }
}

struct TcParams {
  TreeDev tree;
  int32_t n_items, B, H, T;
  int32_t Hk;  // q/k heads (grouped key heads); H when not grouped
  const float* alpha;
  Str3 gate;   // strides of alpha (dense layouts)
  float* O;
  int32_t* status;
  // The tensor maps are 4-D, (channel, node, head, layer*request) or (channel, head, node, ...)
  // whichever has ascending strides: bit 0 / 1 / 2 set = q,k / v / O take the node coordinate
  // before the head coordinate.
  int32_t node_first;
  // packed forest only: request b owns rows offsets[b] .. offsets[b+1]-1 of every plane of
  // `capacity` rows; T is then the per-request node limit (width of the metadata slabs)
  const int32_t* offsets;
  int32_t capacity;
  FastDiv dH, dB, dG;   // division by H, by B, by the q/k group size H / Hk
};

__device__ __forceinline__ PackedItem packed_item(const TcParams& p, int item) {
  PackedItem r;
  const int lb = (int)fdiv((uint32_t)item, p.dH), h = item - lb * p.H;
  const int l = (int)fdiv((uint32_t)lb, p.dB);
  r.b = lb - l * p.B;
  r.plane_v = l * p.H + h;
  r.plane_qk = l * p.Hk + (int)fdiv((uint32_t)h, p.dG);
  r.row0 = p.offsets[r.b];
  r.n = p.offsets[r.b + 1] - r.row0;
  return r;
}

// Load boxes of q, k, v in three heights: the full box (64 or 128 rows), half and a quarter of it.
// A packed forest takes, per request, the smallest that holds its nodes (Section V-B: only the
// tiles inside a request are moved); dense trees always take the full one.
struct LoadMaps {
  CUtensorMap q[3], k[3], v[3];   // [0] quarter, [1] half, [2] full
};
__device__ __forceinline__ int box_class(int n, int full_rows) {
  return n * 4 <= full_rows ? 0 : n * 2 <= full_rows ? 1 : 2;
}

// Coordinates of an item's boxes: (head, outermost) of q/k and of v/O, the first node row, and
// (packed forest) the request's node count.
struct ItemCoord {
  int h_qk, h_v, z, y0, n;
};
template <bool PACKED>
__device__ __forceinline__ ItemCoord item_coord(const TcParams& p, int item) {
  ItemCoord c;
  const int lb = (int)fdiv((uint32_t)item, p.dH), h = item - lb * p.H;
  c.h_v = h;
  c.h_qk = (int)fdiv((uint32_t)h, p.dG);
  if constexpr (PACKED) {
    const int l = (int)fdiv((uint32_t)lb, p.dB), b = lb - l * p.B;
    c.z = l;
    c.y0 = p.offsets[b];
    c.n = p.offsets[b + 1] - c.y0;
  } else {
    c.z = lb;
    c.y0 = 0;
    c.n = p.T;
  }
  return c;
}
// PACKED = packed forest: q/k/v/O are planes of `capacity` rows and an item's rows start at its
// request's offset.  Loads take the fixed box at that offset (rows past the request belong to
// other requests and are masked like padding); stores are cut to the request's node count:
// 8-row-aligned part by TMA boxes of 64/32/16/8 rows (tmO, tmO32, tmO16, tmO8), the last < 8
// rows straight from registers.  The dense instantiation ignores the three extra maps.
// D = dk = dv, 128 or 64.  D = 64 keeps the shared-memory map of D = 128 and uses the first k half,
// the first dv half and the first 64 rows of the state tiles.
template <bool PACKED, bool SMALL, int D>
__global__ void __launch_bounds__(kThreads, 1)
verify_tc_gated_kernel(const __grid_constant__ LoadMaps lm, const __grid_constant__ CUtensorMap tmS,
                       const __grid_constant__ CUtensorMap tmO, const __grid_constant__ CUtensorMap tmO32,
                       const __grid_constant__ CUtensorMap tmO16, const __grid_constant__ CUtensorMap tmO8,
                       const TcParams p) {
  using L = Lay<SMALL>;
  constexpr uint32_t kBox = L::kBox;
  constexpr int kBoxRows = SMALL ? 64 : 128;
  constexpr int NH = D / 64;    // 64-wide halves of a q / k / v row
  constexpr int NC = D / 32;    // 32-float chunks of a state row and of an output row
  constexpr uint32_t kIdescPrefix = idesc_bf16(D, false), kIdescReadout = idesc_bf16(D, true);
  // STACK (T <= 64, D = 128): the hi and lo tiles of a k half lie one behind the other, so one
  // MMA with N = 256 multiplies q by both -- half as many prefix MMAs, each twice as large (an MMA
  // costs about as much to issue whatever its N).  Its 256 columns are one accumulator,
  // q S_hi^T in the first 128 (the readout adds C' V there) and q S_lo^T in the second; the output
  // epilogue adds the two.  TMEM then holds one accumulator, not two: the prefix MMA of item
  // n+1 waits for the output of item n to be read, which it can (it runs under the C' epilogue).
  constexpr bool STACK = SMALL && D == 128;
  constexpr uint32_t kColAccS = 192;   // columns 192..447
  constexpr uint32_t kIdescStack = idesc_bf16(256, false);
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* sm = smem_raw;
  const uint32_t sbase = smem_u32(sm);
  if (sbase & 1023u) {   // the swizzled tiles need this alignment; refuse rather than compute garbage
    if (threadIdx.x == 0 && p.status) atomicExch(p.status, (int)TV_ERR_CUDA);
    return;
  }
  constexpr int kNodes = (int)L::kNodes;
  float* g_s = reinterpret_cast<float*>(sm + L::kOffG);     // [2][kNodes]
  float* f_s = reinterpret_cast<float*>(sm + L::kOffF);     // [2][kNodes]
  float* la_s = reinterpret_cast<float*>(sm + L::kOffAl);   // [kNodes], decay warp only
  volatile int* fast_s = reinterpret_cast<volatile int*>(sm + L::kOffMisc + 16);   // [2]: every |g| <= 100
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + L::kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + L::kOffMisc + 4);
  auto bar = [&](int i) { return sbase + L::kOffBar + 8u * i; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int T = p.T;
  const int n_jh = (!SMALL && T > 64) ? 2 : 1;  // 64-wide j halves that hold real nodes
  const bool nf_qk = p.node_first & 1, nf_v = p.node_first & 2, nf_o = p.node_first & 4;
  // stage of S_pre that item `it` of this CTA uses, and the parity of that use
  auto s_stage = [](uint32_t it) -> int { return SMALL ? (int)(it & 1u) : 0; };
  auto s_phase = [](uint32_t it) -> uint32_t { return SMALL ? ((it >> 1) & 1u) : (it & 1u); };

  if (tid == 0) {
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    mbar_init(bar(QK_FULL), 1);  mbar_init(bar(QK_FREE), 1 + kSplitWarps);
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar(S_FULL0 + s), 1);
      mbar_init(bar(S_CONV0 + s), kSplitWarps);
      mbar_init(bar(S_FREE0 + s), 1);
    }
    mbar_init(bar(V_FULL), 1);   mbar_init(bar(V_FREE), 1);
    mbar_init(bar(SC_DONE), 1);  mbar_init(bar(SC_FREE), kComputeWarps);
    mbar_init(bar(QB_READY0), kSplitWarps);
    mbar_init(bar(QB_READY1), kSplitWarps);
    mbar_init(bar(QS_READY0), kComputeWarps);
    mbar_init(bar(QS_READY1), kComputeWarps);
    mbar_init(bar(C_READY), kComputeWarps);
    mbar_init(bar(ACC_DONE0), 1); mbar_init(bar(ACC_DONE1), 1);
    mbar_init(bar(ACC_FREE0), kComputeWarps); mbar_init(bar(ACC_FREE1), kComputeWarps);
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar(META_READY0 + s), 1);
      mbar_init(bar(META_FREE0 + s), kComputeWarps + 1);   // + the MMA issuer
    }
    mbar_init(bar(OST_READY), kComputeWarps);
    mbar_init(bar(OST_FREE), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if constexpr (PACKED) {
    // V rows below a request's box keep what earlier items left there and only ever meet zero
    // coefficients; before the first item they must not hold NaN patterns (0 x NaN is not 0)
    for (uint32_t o = (uint32_t)tid * 16u; o < 2 * kBox; o += kThreads * 16u)
      *reinterpret_cast<uint4*>(sm + L::kOffV + o) = make_uint4(0u, 0u, 0u, 0u);
    fence_async_smem();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // registers: 128 per thread at launch; the compute warps take what the others give up
  if (warp < kFirstComputeWarp) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
  if (warp == 0) {
    // ===================== TMA producer =====================
    // Three independent load streams (q+k, v, S_pre), each in item order and each gated by the
    // barrier that says its buffer is free.  One thread polls the three gates and issues
    // whatever is ready, so that no stream waits for another one's buffer.
    if (lane == 0) {
      int pend_qk = 0, pend_v = 0, pend_s[2] = {0, 0};
      const uint32_t n_it = blockIdx.x < (uint32_t)p.n_items
                                ? ((uint32_t)p.n_items - blockIdx.x + gridDim.x - 1) / gridDim.x : 0u;
      uint32_t i_qk = 0, i_v = 0, i_s = 0, i_sc = SMALL ? 0u : 0xffffffffu;   // T > 64: the MMA issuer keeps the scores
      // T <= 64 polls without parking (test_wait); T > 64, with items twice as long, measured 1 % faster
      // parked in try_wait
      auto poll = [](uint32_t b, uint32_t parity) { return SMALL ? mbar_test(b, parity) : mbar_try(b, parity); };
      const uint64_t dQ = desc_kmajor(sbase + L::kOffQ), dK = desc_kmajor(sbase + L::kOffK);
      // The first state tile is requested before the wait: the state is written by commit kernels
      // and by the caller's own work only, neither of which releases a dependent before it ends, and
      // the library's kernels that do (metadata, verify, Stage 1) release theirs only after their
      // own wait -- so whenever this kernel runs, S_pre is complete.  q, k, v and the gates may be
      // the output of the kernel directly in front (Stage 1) and wait.
      if (n_it > 0) {
        mbar_expect_tx(bar(S_FULL0), NC * D * 128);
#pragma unroll 1
        for (int c = 0; c < NC; ++c)
          tma_load_3d(sbase + L::kOffS + (uint32_t)c * kTile, &tmS, bar(S_FULL0), 32 * c, 0, (int)blockIdx.x);
        pend_s[0] = 1;
        i_s = 1;
      }
      grid_dependency_wait();   // inputs may come from the kernel in front (dependent launch)
      long long t_idle = clock64();
      uint32_t spin = 0;
      while (i_qk < n_it || i_v < n_it || i_s < n_it || (SMALL && i_sc < n_it)) {
        bool progress = false;
        // A fourth stream, not a load: the score MMAs Sc = Q K^T of item i_sc, issued from here the
        // moment q and k have landed and the score columns are free -- the MMA issuer's thread
        // is the busiest of the CTA, and these eight instructions depend on nothing it does.
        if (SMALL && i_sc < n_it && poll(bar(QK_FULL), i_sc & 1) && poll(bar(SC_FREE), (i_sc & 1) ^ 1)) {
          tc_fence_after();
#pragma unroll(SMALL ? 4 : 1)
          for (uint32_t i = 0; i < 4 * NH; ++i) {   // k half i >> 2, 16 contraction indices (32 bytes) per step
            const uint32_t off = ((i >> 2) * kBox + (i & 3u) * 32u) >> 4;
            mma_bf16_ss(tmem + kColSc, dQ + off, dK + off, SMALL ? kIdescKK64 : kIdescKK128, i);
          }
          tc_commit(bar(SC_DONE));
          tc_commit(bar(QK_FREE));
          ++i_sc;
          progress = true;
        }
        // (two stages: the second item's state is not asked for before the first item's operands
        // have landed -- at the start of a launch every CTA's first loads share the memory system)
        if (i_s < n_it && (!SMALL || i_s != 1 || (poll(bar(S_FULL0), 0) && poll(bar(QK_FULL), 0))) &&
            poll(bar(S_FREE0 + s_stage(i_s)), s_phase(i_s) ^ 1)) {
          const int sj = s_stage(i_s);
          const int item = (int)(blockIdx.x + i_s * gridDim.x);
          mbar_expect_tx(bar(S_FULL0 + sj), NC * D * 128);
#pragma unroll 1
          for (int c = 0; c < NC; ++c)
            tma_load_3d(sbase + L::kOffS + (uint32_t)(sj * 4 + c) * kTile, &tmS, bar(S_FULL0 + sj), 32 * c, 0, item);
          pend_s[sj] = 1 + (int)s_phase(i_s);
          ++i_s;
          progress = true;
        }
        if (i_qk < n_it && poll(bar(QK_FREE), (i_qk & 1) ^ 1)) {
          const ItemCoord ic = item_coord<PACKED>(p, (int)(blockIdx.x + i_qk * gridDim.x));
          // rows of the boxes of this item (the tile layout in shared memory does not depend on it)
          const int bc = PACKED ? box_class(ic.n, kBoxRows) : 2;
          const uint32_t box_bytes = kBox >> (2 - bc);
          mbar_expect_tx(bar(QK_FULL), 2 * NH * box_bytes);
#pragma unroll 1
          for (uint32_t i = 0; i < 4; ++i)   // q: k halves 0, 1; k: k halves 0, 1 (consecutive boxes)
            if ((int)(i & 1u) < NH)
              load_box(sbase + L::kOffQ + i * kBox, i < 2 ? &lm.q[bc] : &lm.k[bc], bar(QK_FULL), nf_qk,
                       (int)(i & 1u) * 64, ic.y0, ic.h_qk, ic.z);
          pend_qk = 1 + (int)(i_qk & 1);
          ++i_qk;
          progress = true;
        }
        if (i_v < n_it && poll(bar(V_FREE), (i_v & 1) ^ 1)) {
          const ItemCoord ic = item_coord<PACKED>(p, (int)(blockIdx.x + i_v * gridDim.x));
          const int bc = PACKED ? box_class(ic.n, kBoxRows) : 2;
          const uint32_t box_bytes = kBox >> (2 - bc);
          mbar_expect_tx(bar(V_FULL), NH * box_bytes);
#pragma unroll 1
          for (uint32_t i = 0; i < NH; ++i)
            load_box(sbase + L::kOffV + i * kBox, &lm.v[bc], bar(V_FULL), nf_v, (int)i * 64, ic.y0, ic.h_v, ic.z);
          pend_v = 1 + (int)(i_v & 1);
          ++i_v;
          progress = true;
        }
        if (progress) {
          t_idle = clock64();
          spin = 0;
        } else if ((++spin & 255u) == 0) {   // the same limit as every other wait of the kernel
          if (*abort_flag) break;
          if (clock64() - t_idle > kWaitLimitCycles) {
            *abort_flag = 1;
            break;
          }
        }
      }
      if (*abort_flag) {
        // Leave no copy of ours in flight: wait (bounded) for the last loads issued.
        if (pend_qk) mbar_wait(bar(QK_FULL), pend_qk - 1, abort_flag + 1);
        for (int s2 = 0; s2 < 2; ++s2)
          if (pend_s[s2]) mbar_wait(bar(S_FULL0 + s2), pend_s[s2] - 1, abort_flag + 1);
        if (pend_v) mbar_wait(bar(V_FULL), pend_v - 1, abort_flag + 1);
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    // The loops over the MMAs of a product: unrolled for T <= 64 (rolled, the address arithmetic
    // between two MMAs slowed their issue enough to cost 1.6 us of a 32 us launch), rolled for
    // T > 64, where the items are twice as long and the smaller code measured 4 % faster (the
    // roles of a CTA share one instruction cache).
    if (lane == 0) {
      const uint64_t dS = desc_kmajor(sbase + L::kOffS), dV = desc_mnmajor(sbase + L::kOffV, kBox);
      const uint64_t dChi = desc_kmajor(sbase + L::kOffChi), dClo = desc_kmajor(sbase + L::kOffClo);
      // a list of up to ten waits, 6 bits each: barrier index * 2 + parity, first wait in the low bits
      auto wait_list = [&](uint64_t w, int n) -> bool {
#pragma unroll 1
        for (; n > 0; --n, w >>= 6)
          if (!mbar_wait(bar((int)((w >> 1) & 31u)), (uint32_t)(w & 1u), abort_flag)) return false;
        return true;
      };
      auto W = [](int b, uint32_t parity) -> uint64_t { return (uint64_t)(b * 2) | parity; };
      uint32_t it = 0;
#pragma unroll 1
      for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++it) {
        const uint32_t ph = it & 1;
        const uint32_t acc_col = STACK ? kColAccS : ph ? kColAcc1 : kColAcc0;
        const uint32_t ph2 = (it >> 1) & 1;   // the two accumulators alternate
        const int st = s_stage(it);
        // scores = Q K^T (T <= 64: issued by the producer thread)
        if constexpr (!SMALL) {
          if (!wait_list(W(QK_FULL, ph) | W(SC_FREE, ph ^ 1) << 6, 2)) break;
          tc_fence_after();
          const uint64_t dQ = desc_kmajor(sbase + L::kOffQ), dK = desc_kmajor(sbase + L::kOffK);
#pragma unroll 1
          for (uint32_t i = 0; i < 4 * NH; ++i) {   // k half i >> 2, 16 contraction indices (32 bytes) per step
            const uint32_t off = ((i >> 2) * kBox + (i & 3u) * 32u) >> 4;
            mma_bf16_ss(tmem + kColSc, dQ + off, dK + off, kIdescKK128, i);
          }
          tc_commit(bar(SC_DONE));
          tc_commit(bar(QK_FREE));
        }
        // acc = Q S_pre^T: A = the q rows (packed bf16 in TMEM), B = hi and lo tiles of S_pre
        if (!wait_list(W(S_CONV0 + st, s_phase(it)) | W(QB_READY0 + (int)ph, ph2) << 6 |
                           W(META_READY0 + (int)ph, ph2) << 12, 3)) break;
        // extreme decay only: the compute warps have replaced the q rows by scaled ones
        const bool rescaled = fast_s[ph] == 0;
        mbar_arrive(bar(META_FREE0 + (int)ph));
        if (!wait_list((STACK ? W(ACC_FREE0, ph ^ 1) : W(ACC_FREE0 + (int)ph, ph2 ^ 1)) | W(QS_READY0 + (int)ph, ph2) << 6,
                       rescaled ? 2 : 1)) break;
        tc_fence_after();
        if constexpr (STACK) {
#pragma unroll 4
          for (uint32_t i = 0; i < 8; ++i) {   // k half i >> 2: its hi tile and, right behind it, its lo tile
            const uint32_t off = (((uint32_t)st * 4u + (i >> 2) * 2u) * kTile + (i & 3u) * 32u) >> 4;
            mma_bf16_ts(tmem + acc_col, tmem + kColQb + ph * 64 + (i >> 2) * 32 + (i & 3u) * 8, dS + off,
                        kIdescStack, i);
          }
        } else {
#pragma unroll(SMALL ? 8 * NH : 1)
          for (uint32_t i = 0; i < 8 * NH; ++i) {   // tile i >> 2 of the stage = (k half, hi | lo)
            const uint32_t off = (((uint32_t)st * 4u + (i >> 2)) * kTile + (i & 3u) * 32u) >> 4;
            mma_bf16_ts(tmem + acc_col, tmem + kColQb + ph * 64 + (i >> 3) * 32 + (i & 3u) * 8, dS + off,
                        kIdescPrefix, i);
          }
        }
        tc_commit(bar(S_FREE0 + st));
        // acc += C'_hi V + C'_lo V
        if (!wait_list(W(C_READY, ph) | W(V_FULL, ph) << 6, 2)) break;
        tc_fence_after();
#pragma unroll 1
        for (uint32_t jh = 0; jh < (uint32_t)n_jh; ++jh)   // j half
#pragma unroll(SMALL ? 4 : 1)
          for (uint32_t i = 0; i < 4; ++i) {
            const uint64_t bdesc = dV + (((jh * 4u + i) * 2048u) >> 4);
            const uint32_t off = (jh * kTile + i * 32u) >> 4;
            mma_bf16_ss(tmem + acc_col, dChi + off, bdesc, kIdescReadout, 1);
            mma_bf16_ss(tmem + acc_col, dClo + off, bdesc, kIdescReadout, 1);
          }
        tc_commit(bar(V_FREE));
        tc_commit(bar(STACK ? ACC_DONE0 : ACC_DONE0 + (int)ph));
      }
    }
  } else if (warp == 2) {
    // ===================== output stores =====================
    // The staged chunks of an item leave by TMA once all compute warps have written them
    // (OST_READY); OST_FREE tells them that the chunks have been read.  SMALL: the chunks are
    // not the C' tiles, and OST_FREE phase k says that the store of item k-1 is read (phase 0
    // is given away up front).  Else: phase k = the store of item k.
    if (lane == 0) {
      if (SMALL) mbar_arrive(bar(OST_FREE));
      uint32_t it = 0;
      for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++it) {
        if (!mbar_wait(bar(OST_READY), it & 1, abort_flag)) break;
        const ItemCoord ic = item_coord<PACKED>(p, item);
        if constexpr (PACKED) {
          // groups of 8 rows, largest boxes first; staging rows r.. start on a 1024-byte
          // boundary, so the swizzle phase of a partial box equals that of the full tile
          const PackedItem pk = packed_item(p, item);
          const int full = pk.n & ~7;
          int r = 0;
          auto put = [&](const CUtensorMap* m, int rows_box) {
            while (full - r >= rows_box) {
#pragma unroll
              for (int c = 0; c < NC; ++c)
                store_box(m, sbase + L::kOffStage + c * L::kStageChunk + (uint32_t)r * 128u, nf_o, 32 * c,
                          ic.y0 + r, ic.h_v, ic.z);
              r += rows_box;
            }
          };
          put(&tmO, 64);
          put(&tmO32, 32);
          put(&tmO16, 16);
          put(&tmO8, 8);
        } else {
#pragma unroll
          for (int c = 0; c < NC; ++c)
            store_box(&tmO, sbase + L::kOffStage + c * L::kStageChunk, nf_o, 32 * c, 0, ic.h_v, ic.z);
        }
        tma_store_commit();
        tma_store_wait_read();
        mbar_arrive(bar(OST_FREE));
      }
      tma_store_wait_all();   // our stores are complete before we leave
    }
  } else {
    // ===================== path decay, ahead of the compute warps =====================
    // g_i = sum of log2(alpha_j) over j in Anc(i) + {i}, for every node of the item: lane l takes
    // nodes l, l + 32, ...; the sum runs over the mask bits against log2(alpha) in shared memory.
    // Results of item n go to copy n & 1 of g / exp2(-g) / the range flag.
    grid_dependency_wait();
    uint32_t it = 0;
    for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++it) {
      const int par = (int)(it & 1);
      const uint64_t* mrow;
      const float* arow;
      int64_t astep;
      int Tb;
      if constexpr (PACKED) {
        const PackedItem pk = packed_item(p, item);
        mrow = p.tree.anc + (size_t)pk.b * T * 2;
        arow = p.alpha + (size_t)pk.plane_v * p.capacity + pk.row0;
        astep = 1;
        Tb = pk.n;
      } else {
        const int lb = (int)fdiv((uint32_t)item, p.dH), h = item - lb * p.H;
        const int tb = p.tree.n_trees == 1 ? 0 : lb - (int)fdiv((uint32_t)lb, p.dB) * p.B;
        mrow = p.tree.anc + (size_t)tb * T * 2;
        arow = p.alpha + (int64_t)lb * p.gate.b + (int64_t)h * p.gate.h;
        astep = p.gate.t;
        Tb = T;
      }
      constexpr int kRows = kNodes / 32;   // nodes per lane
      constexpr int kNone = 255;
      float sum[kRows];   // log2(alpha) summed over the path from the node up to, not including, `up`
      int up[kRows];      // how far that path reaches: an ancestor, or kNone once it is past the root
#pragma unroll
      for (int k = 0; k < kRows; ++k) {
        const int r = k * 32 + lane;
        sum[k] = 1.f;   // the gate for now; rows past the item: log2 = 0
        up[k] = kNone;
        if (r < Tb) {
          sum[k] = arow[(int64_t)r * astep];
          // parents precede their children, so the parent is the highest ancestor
          const uint64_t m0 = mrow[2 * r], m1 = mrow[2 * r + 1];
          if (m1) up[k] = 127 - __clzll((long long)m1);
          else if (m0) up[k] = 63 - __clzll((long long)m0);
        }
      }
      // the compute warps are done with this copy (item it - 2)
      if (!mbar_wait_warp(bar(META_FREE0 + par), ((it >> 1) & 1) ^ 1, abort_flag)) break;
      float* gw = g_s + par * kNodes;
      int* up_s = reinterpret_cast<int*>(la_s);
#pragma unroll
      for (int k = 0; k < kRows; ++k) {
        sum[k] = log2f(sum[k]);
        gw[k * 32 + lane] = sum[k];
        up_s[k * 32 + lane] = up[k];
      }
      __syncwarp();
      // pointer jumping: every round doubles the length of the summed path; ceil(log2(depth + 1))
      // rounds, whatever the shape of the tree
      while (true) {
        bool open = false;
#pragma unroll
        for (int k = 0; k < kRows; ++k) open = open || up[k] != kNone;
        if (!__any_sync(0xffffffffu, open)) break;
        float add[kRows];
        int nup[kRows];
#pragma unroll
        for (int k = 0; k < kRows; ++k) {
          add[k] = 0.f;
          nup[k] = kNone;
          if (up[k] != kNone) {
            add[k] = gw[up[k]];
            nup[k] = up_s[up[k]];
          }
        }
        __syncwarp();
#pragma unroll
        for (int k = 0; k < kRows; ++k) {
          if (up[k] != kNone) {
            sum[k] += add[k];
            up[k] = nup[k];
            gw[k * 32 + lane] = sum[k];
            up_s[k * 32 + lane] = nup[k];
          }
        }
        __syncwarp();
      }
      bool in_range = true;
#pragma unroll
      for (int k = 0; k < kRows; ++k) {
        f_s[par * kNodes + k * 32 + lane] = exp2f(-sum[k]);
        in_range = in_range && fabsf(sum[k]) <= 100.f;
      }
      // exp2(e_i - g_j) = 2^e_i * 2^-g_j is safe when every |g| <= 100; otherwise exp2 is taken per pair
      const bool fast = __all_sync(0xffffffffu, in_range);
      if (lane == 0) fast_s[par] = fast;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(META_READY0 + par));
    }
  }
  } else if (warp >= kFirstSplitWarp) {
    // ===================== operand warps: q rows into TMEM, state split =====================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 104;");
    const int row = tid - kFirstSplitWarp * 32;   // state row v, and node i for the q copy
    const int pw = warp - kFirstSplitWarp;        // = TMEM lane window of this warp
    const uint32_t lane_addr = (uint32_t)(pw * 32) << 16;
    const uint32_t swz = (uint32_t)(row & 7);
    uint32_t it = 0;
    for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++it) {
      const uint32_t ph = it & 1;
      const int st = s_stage(it);
      // ---- q rows (bf16, swizzled boxes) -> TMEM as they are: the A operand of the prefix MMA.
      // Copy it & 1, last read by the prefix MMA of item it - 2.  Two stages: that MMA freed the
      // stage this item now uses.  One stage: the state of item it - 1, already seen here, was
      // only loaded after that MMA had freed the stage.
      auto copy_q = [&]() -> bool {
        if (SMALL && it >= 2 && !mbar_wait_warp(bar(S_FREE0 + st), s_phase(it - 2), abort_flag)) return false;
        if (!mbar_wait_warp(bar(QK_FULL), ph, abort_flag)) return false;
        tc_fence_after();
        if (pw * 32 < T) {
#pragma unroll
          for (int half = 0; half < NH; ++half) {
            const unsigned char* qrow = sm + L::kOffQ + half * kBox + row * 128;
            uint32_t r[32];
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              const uint4 x = *reinterpret_cast<const uint4*>(qrow + (((uint32_t)c ^ swz) << 4));
              r[c * 4 + 0] = x.x; r[c * 4 + 1] = x.y; r[c * 4 + 2] = x.z; r[c * 4 + 3] = x.w;
            }
            tmem_st32(tmem + lane_addr + kColQb + ph * 64 + half * 32, r);
          }
          tmem_wait_st();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(bar(QB_READY0 + (int)ph));
          mbar_arrive(bar(QK_FREE));
        }
        return true;
      };
      // ---- the state split ----
      auto split_state = [&]() -> bool {
        if (!mbar_wait_warp(bar(S_FULL0 + st), s_phase(it), abort_flag)) return false;
        unsigned char* s_buf = sm + L::kOffS + (uint32_t)st * 4u * kTile;
        if (row < D) {   // state rows v < dv
#pragma unroll 1
          for (int half = 0; half < NH; ++half) split_state_row(s_buf, row, half, swz);   // one copy of the code
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(S_CONV0 + st));
        return true;
      };
      // q first: its buffer is single, and the sooner it is free the sooner the next item's q and k
      // are asked for (the split first measured 0.9 us slower per 64-node launch)
      if (!copy_q() || !split_state()) break;
    }
  } else {
    // ===================== compute warps =====================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 168;");
    const int cw = warp - kFirstComputeWarp;
    const int quad = warp & 3;          // TMEM lane window of this warp
    const int hc = cw >> 2;             // column half handled by this warp
    const int row = quad * 32 + lane;   // node i (and state row v in the split of S_pre)
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t swz = (uint32_t)(row & 7);
    const bool warp_live = quad * 32 < T;   // this warp's 32 rows hold at least one node

    // O_i = r_i acc_i for the item whose accumulator is `it_prev`: TMEM -> registers -> four
    // [rows][32 fp32] swizzled staging chunks -> one TMA store per chunk (full 128-byte lines;
    // rows past T are clipped by the tensor map).  SMALL: staging never collides with the C'
    // tiles of the next item and the store is only waited for one item later.  Else: the
    // chunks are the four C' tiles themselves and the store must have read them before C' is
    // rewritten.
    auto final_epilogue = [&](uint32_t it_prev, float r_prev, uint32_t ost_phase, const PackedItem& pk_prev) -> bool {
      const int acc_done = STACK ? ACC_DONE0 : (it_prev & 1) ? ACC_DONE1 : ACC_DONE0;
      const int acc_free = STACK ? ACC_FREE0 : (it_prev & 1) ? ACC_FREE1 : ACC_FREE0;
      const uint32_t acc_col = STACK ? kColAccS : (it_prev & 1) ? kColAcc1 : kColAcc0;
      // SMALL: the store of the item before has read the staging chunks
      if (SMALL && !mbar_wait_warp(bar(OST_FREE), ost_phase, abort_flag)) return false;
      if (!mbar_wait_warp(bar(acc_done), STACK ? (it_prev & 1) : (it_prev >> 1) & 1, abort_flag)) return false;
      tc_fence_after();
      if (warp_live) {
#pragma unroll
        for (int half = 0; half < NH; ++half) {   // this warp's D / 2 columns, 32 at a time
          uint32_t r1[32];
          tmem_ld32(tmem + lane_addr + acc_col + hc * (D / 2) + half * 32, r1);
          if constexpr (STACK) {   // + q S_lo^T from the second half of the accumulator
            uint32_t r2[32];
            tmem_ld32(tmem + lane_addr + acc_col + 128 + hc * 64 + half * 32, r2);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) r1[e] = __float_as_uint(__uint_as_float(r1[e]) + __uint_as_float(r2[e]));
          }
          tmem_wait_ld();
          unsigned char* orow = sm + L::kOffStage + (hc * NH + half) * L::kStageChunk + row * 128;
          // packed forest: the rows after the last full group of 8 leave from registers
          const bool tail_row = PACKED && row >= (pk_prev.n & ~7) && row < pk_prev.n;
          float* otail = nullptr;
          if constexpr (PACKED)
            otail = p.O + ((size_t)pk_prev.plane_v * p.capacity + pk_prev.row0 + row) * D + hc * (D / 2) + half * 32;
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
      return SMALL ? true : mbar_wait_warp(bar(OST_FREE), ost_phase, abort_flag);
    };

    // metadata of the first item; later items are fetched one item ahead
    uint64_t nm0 = 0, nm1 = 0;
    PackedItem npk = {0, 0, 0, 0, T};   // packed forest: rows of the next item
    auto fetch_meta = [&](int item) {
      nm0 = 0; nm1 = 0;
      if constexpr (PACKED) {
        if (item < p.n_items) {
          npk = packed_item(p, item);
          if (row < npk.n) {
            const uint64_t* m = p.tree.anc + ((size_t)npk.b * T + row) * 2;
            nm0 = m[0];
            nm1 = m[1];
          }
        }
      } else if (item < p.n_items && row < T) {
        const int lb = (int)fdiv((uint32_t)item, p.dH);
        const int tb = p.tree.n_trees == 1 ? 0 : lb - (int)fdiv((uint32_t)lb, p.dB) * p.B;
        const uint64_t* m = p.tree.anc + ((size_t)tb * T + row) * 2;
        nm0 = m[0];
        nm1 = m[1];
      }
    };
    // dependent launch: barrier set-up and the TMEM allocation above ran under the tail of the
    // kernel in front; everything that reads global memory waits for it here
    grid_dependency_wait();
    // the commit kernel behind this one may be scheduled as SMs drain (it orders itself)
    if (warp == kFirstComputeWarp && lane == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    fetch_meta(blockIdx.x);

    uint32_t it = 0;
    bool ok = true;
    float r_prev = 0.f;
    PackedItem pk = npk, pk_prev = npk;
    const int total_rows = PACKED ? p.offsets[p.B] : 0;   // rows at and past this one hold no node
    // One pass more than the CTA has items: the last one only writes out the last item (the
    // output code exists once).
#pragma unroll 1
    for (int item = blockIdx.x;; item += gridDim.x, ++it) {
      const bool live = item < p.n_items;
      const uint32_t ph = it & 1;
      const int par = (int)ph;
      uint64_t m0 = nm0, m1 = nm1;
      pk = npk;
      const int Tb = PACKED ? pk.n : T;   // real nodes of this item
      const float* gs = g_s + par * kNodes;
      const float* fs = f_s + par * kNodes;
      bool fast = true;
      float e_int = 0.f, r_scale = 0.f;
      if (live) {
      fetch_meta(item + (int)gridDim.x);   // next item's masks ride under this item's work
      if (row < Tb) {
        if (row < 64) m0 |= 1ull << row; else m1 |= 1ull << (row - 64);   // M+ = M- + I
      }
      // ---- path decay g, exp2(-g) and the range flag of this item: written by the decay warp ----
      if (!(ok = mbar_wait_warp(bar(META_READY0 + par), (it >> 1) & 1, abort_flag))) break;
      const float g = row < Tb ? gs[row] : 0.f;
      fast = fast_s[par] != 0;
      // Row scaling.  Plain form (every |g| <= 100): the accumulator holds  q_i S_pre^T +
      // sum_j 2^(-g_j) s_ij v_j  and O_i = 2^(g_i) acc.  Extreme decay: a row exponent e =
      // round(g_i) keeps every factor in range: the accumulator holds  2^e (q_i S_pre^T) +
      // sum_j 2^(e - g_j) s_ij v_j  and O_i = 2^(g_i - e) acc; e is an integer, so the scaled q
      // stays exact in bf16, and the exponents e - g_j = (e - g_i) + (g_i - g_j) stay small on
      // ancestor pairs.  Below 2^-100 the prefix term is under fp32 resolution of anything it
      // is added to and is dropped.
      const bool tiny = !fast && g < -100.f;
      e_int = fast ? 0.f : (tiny ? g : fminf(rintf(g), 100.f));
      const float a_scale = tiny ? 0.f : exp2f(e_int);
      r_scale = exp2f(g - e_int);
      if (!fast) {
        // extreme decay: replace the q rows that the operand warps copied to TMEM by scaled ones
        if (!(ok = mbar_wait_warp(bar(QB_READY0 + (int)ph), (it >> 1) & 1, abort_flag))) break;
        tc_fence_after();
        if (warp_live && hc < NH) {
          uint32_t r[32];
          tmem_ld32(tmem + lane_addr + kColQb + ph * 64 + hc * 32, r);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e)   // power-of-two scaling: the products are exact in bf16
            r[e] = __byte_perm(__float_as_uint(a_scale * __uint_as_float(r[e] << 16)),
                               __float_as_uint(a_scale * __uint_as_float(r[e] & 0xffff0000u)), 0x7632);
          tmem_st32(tmem + lane_addr + kColQb + ph * 64 + hc * 32, r);
          tmem_wait_st();
        }
        tc_fence_before();
      }
      __syncwarp();
      // (one barrier per copy of q: an arrival for item n + 2 comes after the scores of item
      // n + 1, which the MMA issuer commits after it is through with this one)
      if (lane == 0) mbar_arrive(bar(QS_READY0 + (int)ph));
      }
      // ---- output rows of the previous item: its accumulator is complete once its readout MMA
      // is, and (T > 64) the C' tiles it frees double as the staging area of the output store.
      // Taken before the scores of this item are waited for: they are computed meanwhile. ----
      if (it > 0 && !(ok = final_epilogue(it - 1, r_prev, (it - 1) & 1, pk_prev))) break;
      if (!live) break;
      // ---- scores of this item ----
      if (!(ok = mbar_wait_warp(bar(SC_DONE), ph, abort_flag))) break;
      tc_fence_after();
      if (warp_live) {
        // this warp covers 32 n_jh of the 64 n_jh real columns, 32 at a time
        for (int h = 0; h < n_jh; ++h) {
          const int cbase = hc * 32 * n_jh + h * 32;     // first column j of this group
          uint32_t r[32];
          tmem_ld32(tmem + lane_addr + kColSc + cbase, r);
          tmem_wait_ld();
          const uint32_t bits = cbase < 64 ? (uint32_t)(m0 >> cbase) : (uint32_t)(m1 >> (cbase - 64));
          unsigned char* chi = sm + L::kOffChi + (cbase >> 6) * kTile + row * 128;
          unsigned char* clo = sm + L::kOffClo + (cbase >> 6) * kTile + row * 128;
          const int chunk0 = (cbase & 63) >> 3;
          if (fast) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const float4 fa = *reinterpret_cast<const float4*>(fs + cbase + c * 8);
              const float4 fb = *reinterpret_cast<const float4*>(fs + cbase + c * 8 + 4);
              const float f8[8] = {fa.x, fa.y, fa.z, fa.w, fb.x, fb.y, fb.z, fb.w};
              float cv[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const float x = __uint_as_float(r[c * 8 + e]) * f8[e];
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
                const float x = __uint_as_float(r[c * 8 + e]) * exp2f(e_int - gs[cbase + c * 8 + e]);
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
        const int rows_loaded = kBoxRows >> (2 - box_class(pk.n, kBoxRows));
        if (pk.row0 + rows_loaded > total_rows) {
          if (!(ok = mbar_wait_warp(bar(V_FULL), ph, abort_flag))) break;
          if (row >= total_rows - pk.row0 && row < rows_loaded && hc < NH) {
            uint4* vrow = reinterpret_cast<uint4*>(sm + L::kOffV + hc * kBox + row * 128);
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
        mbar_arrive(bar(META_FREE0 + par));   // this copy of g may take item it + 2
      }
      r_prev = r_scale;
      pk_prev = pk;
    }
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
// Gated rule: the correction rows are the values themselves (U = V), widened to float.  One
// thread per 8 channels of a node row; rows addressed through the strides of v and of U.
__global__ void widen_rows_kernel(const __nv_bfloat16* __restrict__ v, float* __restrict__ U, int n_lb, int H, int T,
                                  int groups, Str3 sv, Str3 so) {   // groups = dv / 8
  const size_t n = (size_t)n_lb * H * T * groups;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const int c8 = (int)(i % groups);
    size_t r = i / groups;
    const int t = (int)(r % T);
    r /= T;
    const int h = (int)(r % H);
    const int64_t lb = (int64_t)(r / H);
    const uint4 x = *reinterpret_cast<const uint4*>(v + lb * sv.b + h * sv.h + t * sv.t + c8 * 8);
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
    float4 a, b;
    a.x = __uint_as_float(w[0] << 16); a.y = __uint_as_float(w[0] & 0xffff0000u);
    a.z = __uint_as_float(w[1] << 16); a.w = __uint_as_float(w[1] & 0xffff0000u);
    b.x = __uint_as_float(w[2] << 16); b.y = __uint_as_float(w[2] & 0xffff0000u);
    b.z = __uint_as_float(w[3] << 16); b.w = __uint_as_float(w[3] & 0xffff0000u);
    float4* dst = reinterpret_cast<float4*>(U + lb * so.b + h * so.h + t * so.t + c8 * 8);
    dst[0] = a;
    dst[1] = b;
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
  const bool d128 = a.dk == 128 && a.dv == 128;
  const bool d64 = a.dk == 64 && a.dv == 64 && a.tree.offsets == nullptr;   // dense layouts only
  return a.bf16 && (d128 || d64) && a.rule == TV_GATED && a.T <= 128;
}

int tv_launch_verify_tc(const VerifyArgs& a, int32_t* status, cudaStream_t stream) {
  if (!tv_verify_tc_supports(a)) return TV_ERR_UNSUPPORTED;
  const bool packed = a.tree.offsets != nullptr;
  const bool small = a.T <= 64;
  const uint64_t items = (uint64_t)a.L * a.B * a.H;
  const uint32_t rows = small ? 64 : 128;    // rows of an operand box and of a staged output chunk
  const uint32_t D = (uint32_t)a.dk;         // = dv
  // 4-D views: dense / strided layouts from the resolved strides, packed forests as planes
  NodeView vq, vv, vo;
  if (!packed) {
    const uint64_t lb = (uint64_t)a.L * a.B;
    vq = NodeView{D, (uint64_t)a.T, (uint64_t)a.Hk, lb, a.lay.qk.b, a.lay.qk.h, a.lay.qk.t};
    vv = NodeView{D, (uint64_t)a.T, (uint64_t)a.H, lb, a.lay.v.b, a.lay.v.h, a.lay.v.t};
    vo = NodeView{D, (uint64_t)a.T, (uint64_t)a.H, lb, a.lay.out.b, a.lay.out.h, a.lay.out.t};
  } else {
    const int64_t cap = a.tree.capacity;
    vq = NodeView{128, (uint64_t)cap, (uint64_t)a.Hk, (uint64_t)a.L, (int64_t)a.Hk * cap * 128, cap * 128, 128};
    vv = NodeView{128, (uint64_t)cap, (uint64_t)a.H, (uint64_t)a.L, (int64_t)a.H * cap * 128, cap * 128, 128};
    vo = vv;
  }
  const void* const ptrs[5] = {a.q, a.k, a.v, a.S_pre, a.O};
  const uint64_t key = view_key(vq) * 3 + view_key(vv) * 5 + view_key(vo) * 7 + items;
  int node_first = 0;
  const MapSet* ms = cached_maps(ptrs, key, a.T, (packed ? 4 : 0) | (a.Hk << 8), [&](CUtensorMap* m) {
    return make_map4(&m[0], a.q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, vq, 64, rows) &&
           make_map4(&m[1], a.k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, vq, 64, rows) &&
           make_map4(&m[2], a.v, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, vv, 64, rows) &&
           make_map(&m[3], a.S_pre, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, items, D, D, 32, D) &&
           make_map4(&m[4], a.O, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, vo, 32, packed ? 64 : rows);
  });
  const MapSet* mo = ms;   // packed forest: output boxes of 32, 16 and 8 rows
  if (packed) {
    const void* const optrs[5] = {a.O, nullptr, nullptr, nullptr, nullptr};
    mo = cached_maps(optrs, key, a.T, 5, [&](CUtensorMap* m) {
      return make_map4(&m[0], a.O, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, vo, 32, 32) &&
             make_map4(&m[1], a.O, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, vo, 32, 16) &&
             make_map4(&m[2], a.O, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, vo, 32, 8);
    });
  }
  // packed forest: q, k, v boxes of half and a quarter of the full height
  const MapSet* mh[2] = {ms, ms};
  if (packed) {
    for (int c = 0; c < 2; ++c) {
      const uint32_t r = rows >> (2 - c);
      const void* const lptrs[5] = {a.q, a.k, a.v, nullptr, nullptr};
      mh[c] = cached_maps(lptrs, key, a.T, 6 + c, [&](CUtensorMap* m) {
        return make_map4(&m[0], a.q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, vq, 64, r) &&
               make_map4(&m[1], a.k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, vq, 64, r) &&
               make_map4(&m[2], a.v, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, vv, 64, r);
      });
    }
  }
  if (!ms || !mo || !mh[0] || !mh[1]) return TV_ERR_CUDA;
  LoadMaps lm;
  for (int c = 0; c < 3; ++c) {
    const MapSet* src = c == 2 ? ms : mh[c];
    lm.q[c] = src->map[0];
    lm.k[c] = src->map[1];
    lm.v[c] = src->map[2];
  }
  node_first = (node_first_of(vq) ? 1 : 0) | (node_first_of(vv) ? 2 : 0) | (node_first_of(vo) ? 4 : 0);
  static thread_local int configured_dev = -1;
  static thread_local int sm_count = 0;
  int dev = 0;
  TV_CUDA_TRY(cudaGetDevice(&dev));
  if (configured_dev != dev) {
    TV_CUDA_TRY(cudaFuncSetAttribute(verify_tc_gated_kernel<false, false, 128>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Lay<false>::kSmemBytes));
    TV_CUDA_TRY(cudaFuncSetAttribute(verify_tc_gated_kernel<true, false, 128>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Lay<false>::kSmemBytes));
    TV_CUDA_TRY(cudaFuncSetAttribute(verify_tc_gated_kernel<false, true, 128>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Lay<true>::kSmemBytes));
    TV_CUDA_TRY(cudaFuncSetAttribute(verify_tc_gated_kernel<true, true, 128>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Lay<true>::kSmemBytes));
    TV_CUDA_TRY(cudaFuncSetAttribute(verify_tc_gated_kernel<false, false, 64>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Lay<false>::kSmemBytes));
    TV_CUDA_TRY(cudaFuncSetAttribute(verify_tc_gated_kernel<false, true, 64>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Lay<true>::kSmemBytes));
    TV_CUDA_TRY(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev));
    configured_dev = dev;
  }
  TcParams p;
  p.tree = a.tree;
  p.n_items = (int32_t)items;
  p.B = a.B; p.H = a.H; p.T = a.T; p.Hk = a.Hk;
  p.alpha = a.alpha;
  p.gate = a.lay.gate;
  p.O = a.O;
  p.status = status;
  p.node_first = node_first;
  p.offsets = a.tree.offsets;
  p.capacity = a.tree.capacity;
  p.dH = make_fastdiv((uint32_t)a.H);
  p.dB = make_fastdiv((uint32_t)a.B);
  p.dG = make_fastdiv((uint32_t)(a.H / a.Hk));
  const int grid = (int)(items < (uint64_t)sm_count ? items : (uint64_t)sm_count);
  const size_t smem = small ? Lay<true>::kSmemBytes : Lay<false>::kSmemBytes;
  auto go = [&](auto kernel) {
    return launch_dependent(kernel, grid, kThreads, smem, stream, lm, ms->map[3], ms->map[4], mo->map[packed ? 0 : 4], mo->map[packed ? 1 : 4], mo->map[packed ? 2 : 4], p);
  };
  if (packed) {
    TV_CUDA_TRY(small ? go(verify_tc_gated_kernel<true, true, 128>) : go(verify_tc_gated_kernel<true, false, 128>));
    if (a.U) {
      const size_t planes = (size_t)a.L * a.H;
      widen_bf16_rows_kernel<<<dim3(64, (unsigned)(planes < 65535 ? planes : 65535)), 256, 0, stream>>>(
          reinterpret_cast<const __nv_bfloat16*>(a.v), a.U, planes, (size_t)a.tree.capacity, a.tree.offsets, a.B);
      TV_CUDA_TRY(cudaGetLastError());
    }
    return TV_OK;
  }
  if (D == 64)
    TV_CUDA_TRY(small ? go(verify_tc_gated_kernel<false, true, 64>) : go(verify_tc_gated_kernel<false, false, 64>));
  else
    TV_CUDA_TRY(small ? go(verify_tc_gated_kernel<false, true, 128>) : go(verify_tc_gated_kernel<false, false, 128>));
  if (a.U) {
    const size_t n = items * a.T * (D / 8);
    const int blocks = (int)((n + 255) / 256 < 4096 ? (n + 255) / 256 : 4096);
    widen_rows_kernel<<<blocks, 256, 0, stream>>>(reinterpret_cast<const __nv_bfloat16*>(a.v), a.U, a.L * a.B, a.H,
                                                  a.T, (int)(D / 8), a.lay.v, a.lay.out);
    TV_CUDA_TRY(cudaGetLastError());
  }
  return TV_OK;
}
