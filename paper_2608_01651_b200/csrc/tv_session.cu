// Host-buffer round: the whole hot path (tree_build -> tree_verify ->
// commit_path) for callers whose tensors live in host memory.  A session owns
// the device copies; a round moves the inputs in, runs the same entry points
// a device-resident caller uses, and moves O and S_new out.
#include <new>

#include "tv_internal.h"

struct tv_session {
  tv_dims dims;
  int32_t n_trees = 0;
  tv_tree* tree = nullptr;
  char* d_base = nullptr;
  float *S = nullptr, *alpha = nullptr, *beta = nullptr, *O = nullptr, *U = nullptr;
  void *q = nullptr, *k = nullptr, *v = nullptr;
  int32_t* accepted = nullptr;
  size_t nS = 0, nQ = 0, nV = 0, nG = 0, eb = 0;
};

static size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

#define TV_API __attribute__((visibility("default")))

extern "C" {

TV_API int tv_session_create(const tv_dims* d, int32_t n_trees, tv_session** out) {
  if (!out) return TV_ERR_BAD_ARG;
  *out = nullptr;
  if (!d || (n_trees != 1 && n_trees != d->B)) return TV_ERR_BAD_ARG;
  if (d->L < 1 || d->B < 1 || d->H < 1 || d->T < 1 || d->T > TV_MAX_NODES) return TV_ERR_BAD_ARG;
  tv_session* s = new (std::nothrow) tv_session();
  if (!s) return TV_ERR_NOMEM;
  s->dims = *d;
  s->n_trees = n_trees;
  const size_t items = (size_t)d->L * d->B * d->H;
  s->eb = d->qkv_dtype == TV_BF16 ? 2 : 4;
  s->nS = items * d->dv * d->dk;
  if (d->Hk < 0 || d->Hk > d->H || (d->Hk > 0 && d->H % d->Hk != 0)) {
    delete s;
    return TV_ERR_BAD_ARG;
  }
  s->nQ = (size_t)d->L * d->B * (d->Hk ? d->Hk : d->H) * d->T * d->dk;
  s->nV = items * d->T * d->dv;
  s->nG = items * d->T;
  const bool delta = d->rule == TV_GATED_DELTA;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += up256(bytes); return o; };
  const size_t oS = take(s->nS * 4), oq = take(s->nQ * s->eb), ok = take(s->nQ * s->eb),
               ov = take(s->nV * s->eb), oa = take(s->nG * 4), ob = take(s->nG * 4),
               oO = take(s->nV * 4), oU = take(delta ? s->nV * 4 : 0), oacc = take((size_t)d->B * 4);
  cudaError_t e = cudaMalloc((void**)&s->d_base, off);
  if (e != cudaSuccess) {
    tv_set_cuda_error(e);
    delete s;
    return TV_ERR_CUDA;
  }
  s->S = (float*)(s->d_base + oS);
  s->q = s->d_base + oq;
  s->k = s->d_base + ok;
  s->v = s->d_base + ov;
  s->alpha = (float*)(s->d_base + oa);
  s->beta = delta ? (float*)(s->d_base + ob) : nullptr;
  s->O = (float*)(s->d_base + oO);
  s->U = delta ? (float*)(s->d_base + oU) : nullptr;
  s->accepted = (int32_t*)(s->d_base + oacc);
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
  int st;
  if (!s->tree) st = tv_tree_build(parent, s->n_trees, d.T, &s->tree);
  else st = tv_tree_rebuild(s->tree, parent);
  if (st != TV_OK) return st;
  cudaStream_t cs = (cudaStream_t)stream;
  st = tv_tree_upload(s->tree, stream);
  if (st != TV_OK) return st;
  TV_CUDA_TRY(cudaMemcpyAsync(s->S, S_pre, s->nS * 4, cudaMemcpyHostToDevice, cs));
  TV_CUDA_TRY(cudaMemcpyAsync(s->q, q, s->nQ * s->eb, cudaMemcpyHostToDevice, cs));
  TV_CUDA_TRY(cudaMemcpyAsync(s->k, k, s->nQ * s->eb, cudaMemcpyHostToDevice, cs));
  TV_CUDA_TRY(cudaMemcpyAsync(s->v, v, s->nV * s->eb, cudaMemcpyHostToDevice, cs));
  TV_CUDA_TRY(cudaMemcpyAsync(s->alpha, alpha, s->nG * 4, cudaMemcpyHostToDevice, cs));
  if (delta) TV_CUDA_TRY(cudaMemcpyAsync(s->beta, beta, s->nG * 4, cudaMemcpyHostToDevice, cs));
  TV_CUDA_TRY(cudaMemcpyAsync(s->accepted, accepted, (size_t)d.B * 4, cudaMemcpyHostToDevice, cs));
  st = tv_tree_verify(s->tree, &d, s->S, s->q, s->k, s->v, s->alpha, s->beta, s->O, s->U, stream);
  if (st != TV_OK) return st;
  st = tv_commit_path(s->tree, &d, s->accepted, s->S, s->k, s->v, s->alpha, s->beta, s->U, s->S,
                      stream);
  if (st != TV_OK) return st;
  TV_CUDA_TRY(cudaMemcpyAsync(O, s->O, s->nV * 4, cudaMemcpyDeviceToHost, cs));
  TV_CUDA_TRY(cudaMemcpyAsync(S_new, s->S, s->nS * 4, cudaMemcpyDeviceToHost, cs));
  TV_CUDA_TRY(cudaStreamSynchronize(cs));
  return TV_OK;
}

TV_API int tv_session_free(tv_session* s) {
  if (!s) return TV_OK;
  if (s->tree) tv_tree_free(s->tree);
  if (s->d_base) cudaFree(s->d_base);
  delete s;
  return TV_OK;
}

}  // extern "C"
