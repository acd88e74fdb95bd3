// Host-buffer round: the whole hot path (tree_build -> tree_verify ->
// commit_path) for callers whose tensors live in host memory.  A session owns
// the device copies; a round moves the inputs in, runs the same entry points
// a device-resident caller uses, and moves O and S_new out, group of requests
// by group of requests so that transfers and kernels overlap.
#include <new>

#include "tv_internal.h"

// The batch is cut into up to kMaxChunks groups of requests that flow through three internal
// streams -- copies in, kernels, copies out -- chained by one event per group and stage: the
// host->device engine runs through all groups without a pause, a group's kernels start when its
// inputs have landed, and its outputs leave (on the other copy engine) while later groups are
// still arriving.  What is not overlapped is one group's kernels and its copy out: the more
// groups, the shorter that tail.  Requests are independent (Section IV-B), so the groups need no
// exchange.
constexpr int kMaxChunks = 8;

struct tv_chunk {
  int32_t b0 = 0, nb = 0;     // requests [b0, b0 + nb)
  tv_tree* tree = nullptr;
  float *S = nullptr, *alpha = nullptr, *beta = nullptr, *O = nullptr, *U = nullptr;
  void *q = nullptr, *k = nullptr, *v = nullptr;
  int32_t* accepted = nullptr;
};

struct tv_session {
  tv_dims dims;
  int32_t n_trees = 0, n_chunks = 0;
  tv_chunk chunk[kMaxChunks];
  char* d_base = nullptr;
  size_t eb = 0;
  cudaStream_t side[3] = {nullptr, nullptr, nullptr};   // copies in, kernels, copies out
  cudaEvent_t start = nullptr, done[3] = {nullptr, nullptr, nullptr};
  cudaEvent_t in_done[kMaxChunks] = {}, k_done[kMaxChunks] = {};
};

static size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

#define TV_API __attribute__((visibility("default")))

extern "C" {

TV_API int tv_session_free(tv_session* s);

TV_API int tv_session_create(const tv_dims* d, int32_t n_trees, tv_session** out) {
  if (!out) return TV_ERR_BAD_ARG;
  *out = nullptr;
  if (!d || (n_trees != 1 && n_trees != d->B)) return TV_ERR_BAD_ARG;
  if (d->L < 1 || d->B < 1 || d->H < 1 || d->T < 1 || d->T > TV_MAX_NODES) return TV_ERR_BAD_ARG;
  if (d->Hk < 0 || d->Hk > d->H || (d->Hk > 0 && d->H % d->Hk != 0)) return TV_ERR_BAD_ARG;
  tv_session* s = new (std::nothrow) tv_session();
  if (!s) return TV_ERR_NOMEM;
  s->dims = *d;
  s->n_trees = n_trees;
  s->eb = d->qkv_dtype == TV_BF16 ? 2 : 4;
  const bool delta = d->rule == TV_GATED_DELTA;
  const size_t Hk = d->Hk ? d->Hk : d->H;
  {
    // About 48 MB of traffic (both directions) per group, between 2 and kMaxChunks groups: measured
    // on PCIe 5 x16, smaller groups lose more to per-copy overhead than their shorter tail wins
    // (218 MB per round: 3-6 groups within 1 %; 1.2 GB per round: 8 groups 5 % ahead of 4; with
    // the tapered sizes below 5 groups of 48 MB measured 3 % ahead of 7 groups of 32 MB).
    const size_t per_req = (size_t)d->L * ((size_t)d->H * d->dv * d->dk * 8 + 2 * Hk * d->T * d->dk * s->eb +
                                           (size_t)d->H * d->T * d->dv * (s->eb + 4));
    size_t n = (per_req * d->B + (48u << 20) - 1) / (48u << 20);
    n = n < 2 ? 2 : n > (size_t)kMaxChunks ? (size_t)kMaxChunks : n;
    s->n_chunks = (size_t)d->B < n ? d->B : (int32_t)n;
  }
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += up256(bytes); return o; };
  size_t o[kMaxChunks][9];
  for (int c = 0; c < s->n_chunks; ++c) {
    tv_chunk& ch = s->chunk[c];
    // Group sizes rise to the middle and fall again (1 : 2 : 3 : 2 : 1 ...): the first group's
    // copy in and the last group's copy out are the two stretches of a round in which only one
    // direction of the link is busy, so those two groups are the small ones.
    auto cum = [&](int upto) {   // sum of the weights of groups 0 .. upto-1, weight_i = min(i, n-1-i) + 1
      int64_t t = 0;
      for (int i = 0; i < upto; ++i) t += (i < s->n_chunks - 1 - i ? i : s->n_chunks - 1 - i) + 1;
      return t;
    };
    const int64_t wsum = cum(s->n_chunks);
    auto bound = [&](int upto) {   // first request of group `upto`: every group keeps at least one request
      int64_t b = ((int64_t)d->B * cum(upto) + wsum / 2) / wsum;
      if (b < upto) b = upto;
      if (b > d->B - (s->n_chunks - upto)) b = d->B - (s->n_chunks - upto);
      return (int32_t)b;
    };
    ch.b0 = bound(c);
    ch.nb = bound(c + 1) - ch.b0;
    const size_t items = (size_t)d->L * ch.nb * d->H, qitems = (size_t)d->L * ch.nb * Hk;
    o[c][0] = take(items * d->dv * d->dk * 4);
    o[c][1] = take(qitems * d->T * d->dk * s->eb);
    o[c][2] = take(qitems * d->T * d->dk * s->eb);
    o[c][3] = take(items * d->T * d->dv * s->eb);
    o[c][4] = take(items * d->T * 4);
    o[c][5] = take(items * d->T * 4);
    o[c][6] = take(items * d->T * d->dv * 4);
    o[c][7] = take(delta ? items * d->T * d->dv * 4 : 0);
    o[c][8] = take((size_t)ch.nb * 4);
  }
  cudaError_t e = cudaMalloc((void**)&s->d_base, off);
  for (int i = 0; i < 3 && e == cudaSuccess; ++i) {
    e = cudaStreamCreateWithFlags(&s->side[i], cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s->done[i], cudaEventDisableTiming);
  }
  for (int c = 0; c < s->n_chunks && e == cudaSuccess; ++c) {
    e = cudaEventCreateWithFlags(&s->in_done[c], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s->k_done[c], cudaEventDisableTiming);
  }
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s->start, cudaEventDisableTiming);
  if (e != cudaSuccess) {
    tv_set_cuda_error(e);
    tv_session_free(s);
    return TV_ERR_CUDA;
  }
  for (int c = 0; c < s->n_chunks; ++c) {
    tv_chunk& ch = s->chunk[c];
    ch.S = (float*)(s->d_base + o[c][0]);
    ch.q = s->d_base + o[c][1];
    ch.k = s->d_base + o[c][2];
    ch.v = s->d_base + o[c][3];
    ch.alpha = (float*)(s->d_base + o[c][4]);
    ch.beta = delta ? (float*)(s->d_base + o[c][5]) : nullptr;
    ch.O = (float*)(s->d_base + o[c][6]);
    ch.U = delta ? (float*)(s->d_base + o[c][7]) : nullptr;
    ch.accepted = (int32_t*)(s->d_base + o[c][8]);
  }
  *out = s;
  return TV_OK;
}

TV_API int tv_session_round(tv_session* s, const int32_t* parent, const int32_t* accepted,
                            const float* S_pre, const void* q, const void* k, const void* v,
                            const float* alpha, const float* beta, float* O, float* S_new,
                            void* stream) {
  if (!s || !parent || !accepted || !S_pre || !q || !k || !v || !alpha || !O || !S_new)
    return TV_ERR_BAD_ARG;
  const tv_dims& d = s->dims;
  const bool delta = d.rule == TV_GATED_DELTA;
  if (delta && !beta) return TV_ERR_BAD_ARG;
  for (int b = 0; b < d.B; ++b)
    if (accepted[b] < -1 || accepted[b] >= d.T) return TV_ERR_BAD_ARG;
  // malformed trees are refused before anything is queued
  for (size_t t = 0; t < (size_t)s->n_trees; ++t)
    for (int i = 0; i < d.T; ++i) {
      const int32_t p = parent[t * d.T + i];
      if (p < -1 || p >= i) return TV_ERR_INVALID_TREE;
    }
  const size_t Hk = d.Hk ? d.Hk : d.H;
  // bytes of one request of one layer in each tensor
  const size_t rS = (size_t)d.H * d.dv * d.dk * 4, rQ = Hk * d.T * d.dk * s->eb, rV = (size_t)d.H * d.T * d.dv * s->eb,
               rG = (size_t)d.H * d.T * 4, rO = (size_t)d.H * d.T * d.dv * 4;
  cudaStream_t user = (cudaStream_t)stream;
  TV_CUDA_TRY(cudaEventRecord(s->start, user));
  for (int i = 0; i < 3; ++i) TV_CUDA_TRY(cudaStreamWaitEvent(s->side[i], s->start, 0));
  cudaStream_t in = s->side[0], cs = s->side[1], out = s->side[2];
  // From here on copies to and from the caller's host buffers may be in flight: an error return
  // first waits for everything already queued on the three streams, so that the caller never
  // gets control back (and never frees the session) under running work.
  auto fail = [&](int status) {
    for (int i = 0; i < 3; ++i) cudaStreamSynchronize(s->side[i]);
    return status;
  };
#define TV_ROUND_TRY(expr)                \
  do {                                    \
    cudaError_t e__ = (expr);             \
    if (e__ != cudaSuccess) {             \
      tv_set_cuda_error(e__);             \
      return fail(TV_ERR_CUDA);           \
    }                                     \
  } while (0)
  for (int c = 0; c < s->n_chunks; ++c) {
    tv_chunk& ch = s->chunk[c];
    const int32_t* par = s->n_trees == 1 ? parent : parent + (size_t)ch.b0 * d.T;
    const int32_t nt = s->n_trees == 1 ? 1 : ch.nb;
    int st = ch.tree ? tv_tree_rebuild(ch.tree, par) : tv_tree_build(par, nt, d.T, &ch.tree);
    if (st != TV_OK) return fail(st);
    auto h2d = [&](void* dst, const void* src, size_t per_req) -> cudaError_t {
      for (int l = 0; l < d.L; ++l) {   // the group's requests are contiguous within a layer
        cudaError_t e = cudaMemcpyAsync((char*)dst + (size_t)l * ch.nb * per_req,
                                        (const char*)src + ((size_t)l * d.B + ch.b0) * per_req,
                                        (size_t)ch.nb * per_req, cudaMemcpyHostToDevice, in);
        if (e != cudaSuccess) return e;
      }
      return cudaSuccess;
    };
    TV_ROUND_TRY(h2d(ch.S, S_pre, rS));
    TV_ROUND_TRY(h2d(ch.q, q, rQ));
    TV_ROUND_TRY(h2d(ch.k, k, rQ));
    TV_ROUND_TRY(h2d(ch.v, v, rV));
    TV_ROUND_TRY(h2d(ch.alpha, alpha, rG));
    if (delta) TV_ROUND_TRY(h2d(ch.beta, beta, rG));
    TV_ROUND_TRY(cudaMemcpyAsync(ch.accepted, accepted + ch.b0, (size_t)ch.nb * 4, cudaMemcpyHostToDevice, in));
    TV_ROUND_TRY(cudaEventRecord(s->in_done[c], in));
    TV_ROUND_TRY(cudaStreamWaitEvent(cs, s->in_done[c], 0));
    st = tv_tree_upload(ch.tree, cs);
    if (st != TV_OK) return fail(st);
    tv_dims dc = d;
    dc.B = ch.nb;
    st = tv_tree_verify(ch.tree, &dc, ch.S, ch.q, ch.k, ch.v, ch.alpha, ch.beta, ch.O, ch.U, cs);
    if (st != TV_OK) return fail(st);
    st = tv_commit_path(ch.tree, &dc, ch.accepted, ch.S, ch.k, ch.v, ch.alpha, ch.beta, ch.U, ch.S, cs);
    if (st != TV_OK) return fail(st);
    TV_ROUND_TRY(cudaEventRecord(s->k_done[c], cs));
    TV_ROUND_TRY(cudaStreamWaitEvent(out, s->k_done[c], 0));
    for (int l = 0; l < d.L; ++l) {
      TV_ROUND_TRY(cudaMemcpyAsync((char*)O + ((size_t)l * d.B + ch.b0) * rO, (char*)ch.O + (size_t)l * ch.nb * rO,
                                  (size_t)ch.nb * rO, cudaMemcpyDeviceToHost, out));
      TV_ROUND_TRY(cudaMemcpyAsync((char*)S_new + ((size_t)l * d.B + ch.b0) * rS,
                                  (char*)ch.S + (size_t)l * ch.nb * rS, (size_t)ch.nb * rS,
                                  cudaMemcpyDeviceToHost, out));
    }
  }
  for (int i = 0; i < 3; ++i) {
    TV_ROUND_TRY(cudaEventRecord(s->done[i], s->side[i]));
    TV_ROUND_TRY(cudaStreamWaitEvent(user, s->done[i], 0));
  }
  TV_ROUND_TRY(cudaStreamSynchronize(user));
  return TV_OK;
#undef TV_ROUND_TRY
}

TV_API int tv_session_free(tv_session* s) {
  if (!s) return TV_OK;
  for (int c = 0; c < kMaxChunks; ++c)
    if (s->chunk[c].tree) tv_tree_free(s->chunk[c].tree);
  for (int i = 0; i < 3; ++i) {
    if (s->side[i]) cudaStreamDestroy(s->side[i]);
    if (s->done[i]) cudaEventDestroy(s->done[i]);
  }
  for (int c = 0; c < kMaxChunks; ++c) {
    if (s->in_done[c]) cudaEventDestroy(s->in_done[c]);
    if (s->k_done[c]) cudaEventDestroy(s->k_done[c]);
  }
  if (s->start) cudaEventDestroy(s->start);
  if (s->d_base) cudaFree(s->d_base);
  delete s;
  return TV_OK;
}

}  // extern "C"
