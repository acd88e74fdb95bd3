// C ABI of libtreeverify: host-side tree metadata, argument validation, dispatch.
#include <cstring>
#include <new>

#include "tv_internal.h"

static thread_local int g_last_cuda_error = 0;
void tv_set_cuda_error(cudaError_t e) { g_last_cuda_error = (int)e; }

#define TV_API __attribute__((visibility("default")))

extern "C" {

TV_API const char* tv_strerror(int s) {
  switch (s) {
    case TV_OK: return "ok";
    case TV_ERR_BAD_ARG: return "bad argument (null or misaligned pointer, or size out of range)";
    case TV_ERR_INVALID_TREE: return "invalid tree (need -1 <= parent[i] < i)";
    case TV_ERR_UNSUPPORTED: return "unsupported shape, dtype or rule";
    case TV_ERR_CUDA: return "CUDA runtime error (see tv_last_cuda_error)";
    case TV_ERR_NOT_UPLOADED: return "tree metadata not uploaded to the device";
    case TV_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case TV_ERR_NOMEM: return "out of memory";
    case TV_ERR_TOO_LARGE: return "size beyond the fixed capacity of this entry point";
    default: return "unknown status";
  }
}

TV_API int tv_version(void) { return 100; }
TV_API int tv_last_cuda_error(void) { return g_last_cuda_error; }

// ---------------------------------------------------------------------------
// Tree metadata.  Nodes are indexed parent before child, so one forward sweep
// gives every strict-ancestor set: anc(i) = anc(parent(i)) + {parent(i)}.
// ---------------------------------------------------------------------------
static int fill_tree(tv_tree* t, const int32_t* parent) {
  const int n = t->n;
  int md_all = 0;
  for (int tr = 0; tr < t->n_trees; ++tr) {
    const int32_t* par = parent + (size_t)tr * n;
    for (int i = 0; i < n; ++i)
      if (par[i] < -1 || par[i] >= i) return TV_ERR_INVALID_TREE;
  }
  for (int tr = 0; tr < t->n_trees; ++tr) {
    const int32_t* par = parent + (size_t)tr * n;
    uint64_t* anc = t->anc.data() + (size_t)tr * n * 2;
    int32_t* dep = t->depth.data() + (size_t)tr * n;
    int md = 0;
    for (int i = 0; i < n; ++i) {
      const int p = par[i];
      uint64_t w0 = 0, w1 = 0;
      int d = 0;
      if (p >= 0) {
        w0 = anc[2 * p];
        w1 = anc[2 * p + 1];
        if (p < 64) w0 |= (uint64_t)1 << p; else w1 |= (uint64_t)1 << (p - 64);
        d = dep[p] + 1;
      }
      anc[2 * i] = w0;
      anc[2 * i + 1] = w1;
      dep[i] = d;
      if (d > md) md = d;
    }
    t->max_depth[tr] = md;
    if (md > md_all) md_all = md;
  }
  std::memcpy(t->parent.data(), parent, sizeof(int32_t) * (size_t)t->n_trees * n);
  t->max_depth_all = md_all;
  t->uploaded = false;
  t->host_meta_valid = true;
  return TV_OK;
}

TV_API int tv_tree_build(const int32_t* parent, int32_t n_trees, int32_t n, tv_tree** out) {
  if (!out) return TV_ERR_BAD_ARG;
  *out = nullptr;
  if (!parent || n_trees < 1 || n < 1) return TV_ERR_BAD_ARG;
  if (n > TV_MAX_NODES) return TV_ERR_UNSUPPORTED;
  tv_tree* t = new (std::nothrow) tv_tree();
  if (!t) return TV_ERR_NOMEM;
  t->n_trees = n_trees;
  t->n = n;
  try {
    t->parent.resize((size_t)n_trees * n);
    t->depth.resize((size_t)n_trees * n);
    t->max_depth.resize(n_trees);
    t->anc.resize((size_t)n_trees * n * 2);
  } catch (...) {
    delete t;
    return TV_ERR_NOMEM;
  }
  int st = fill_tree(t, parent);
  if (st != TV_OK) {
    delete t;
    return st;
  }
  *out = t;
  return TV_OK;
}

TV_API int tv_tree_rebuild(tv_tree* t, const int32_t* parent) {
  if (!t || !parent) return TV_ERR_BAD_ARG;
  if (!t->offsets.empty()) return TV_ERR_BAD_ARG;   // a packed forest is rebuilt with its offsets
  return fill_tree(t, parent);
}

// Packed forest: the flat parent array is spread into per-tree slabs of n entries (padding =
// root children nobody descends from), so all metadata code above and every kernel's mask
// handling serve both layouts; only the tensor rows are packed.
static int fill_forest(tv_tree* t, const int32_t* parent_flat, const int32_t* offsets) {
  const int B = t->n_trees, n = t->n;
  if (offsets[0] != 0) return TV_ERR_BAD_ARG;
  for (int b = 0; b < B; ++b) {
    const int nb = offsets[b + 1] - offsets[b];
    if (nb < 1 || nb > n) return TV_ERR_BAD_ARG;
  }
  if (offsets[B] > t->capacity) return TV_ERR_TOO_LARGE;
  std::vector<int32_t> padded;
  try {
    padded.assign((size_t)B * n, -1);
  } catch (...) {
    return TV_ERR_NOMEM;
  }
  for (int b = 0; b < B; ++b)
    std::memcpy(padded.data() + (size_t)b * n, parent_flat + offsets[b],
                sizeof(int32_t) * (size_t)(offsets[b + 1] - offsets[b]));
  int st = fill_tree(t, padded.data());
  if (st != TV_OK) return st;
  std::memcpy(t->offsets.data(), offsets, sizeof(int32_t) * (size_t)(B + 1));
  return TV_OK;
}

TV_API int tv_forest_build(const int32_t* parent_flat, const int32_t* offsets, int32_t n_req, int32_t n_max,
                           int32_t capacity, tv_tree** out) {
  if (!out) return TV_ERR_BAD_ARG;
  *out = nullptr;
  if (!parent_flat || !offsets || n_req < 1 || n_max < 1 || capacity < 1) return TV_ERR_BAD_ARG;
  if (n_max > TV_MAX_NODES) return TV_ERR_UNSUPPORTED;
  tv_tree* t = new (std::nothrow) tv_tree();
  if (!t) return TV_ERR_NOMEM;
  t->n_trees = n_req;
  t->n = n_max;
  t->capacity = capacity;
  try {
    t->parent.resize((size_t)n_req * n_max);
    t->depth.resize((size_t)n_req * n_max);
    t->max_depth.resize(n_req);
    t->anc.resize((size_t)n_req * n_max * 2);
    t->offsets.resize((size_t)n_req + 1);
  } catch (...) {
    delete t;
    return TV_ERR_NOMEM;
  }
  int st = fill_forest(t, parent_flat, offsets);
  if (st != TV_OK) {
    delete t;
    return st;
  }
  *out = t;
  return TV_OK;
}

TV_API int tv_forest_rebuild(tv_tree* t, const int32_t* parent_flat, const int32_t* offsets) {
  if (!t || !parent_flat || !offsets || t->offsets.empty()) return TV_ERR_BAD_ARG;
  return fill_forest(t, parent_flat, offsets);
}

TV_API int tv_tree_meta(const tv_tree* t, uint64_t* anc, int32_t* depth, int32_t* max_depth) {
  if (!t) return TV_ERR_BAD_ARG;
  if (!t->host_meta_valid) return TV_ERR_UNSUPPORTED;   // topology came from the device
  if (anc) std::memcpy(anc, t->anc.data(), t->anc.size() * sizeof(uint64_t));
  if (depth) std::memcpy(depth, t->depth.data(), t->depth.size() * sizeof(int32_t));
  if (max_depth) std::memcpy(max_depth, t->max_depth.data(), t->max_depth.size() * sizeof(int32_t));
  return TV_OK;
}

TV_API int tv_tree_info(const tv_tree* t, int32_t* n_trees, int32_t* n, int32_t* max_depth_all) {
  if (!t) return TV_ERR_BAD_ARG;
  if (n_trees) *n_trees = t->n_trees;
  if (n) *n = t->n;
  if (max_depth_all) *max_depth_all = t->max_depth_all;
  return TV_OK;
}

TV_API int tv_tree_path(const tv_tree* t, const int32_t* accepted, int32_t n_req, int32_t* path,
                 int32_t path_stride, int32_t* len) {
  if (!t || !accepted || !path || !len || n_req < 0) return TV_ERR_BAD_ARG;
  if (!t->host_meta_valid) return TV_ERR_UNSUPPORTED;   // topology came from the device
  if (path_stride < t->max_depth_all + 1) return TV_ERR_BAD_ARG;
  if (t->n_trees != 1 && n_req > t->n_trees) return TV_ERR_BAD_ARG;
  for (int r = 0; r < n_req; ++r)
    if (accepted[r] < -1 || accepted[r] >= t->n) return TV_ERR_BAD_ARG;
  for (int r = 0; r < n_req; ++r) {
    const int tr = t->n_trees == 1 ? 0 : r;
    int32_t* row = path + (size_t)r * path_stride;
    for (int s = 0; s < path_stride; ++s) row[s] = -1;
    const int a = accepted[r];
    if (a < 0) {
      len[r] = 0;
      continue;
    }
    // Indices grow along a root-to-node path, so the set bits of the ancestor
    // mask in increasing order are the path in topological order.
    const uint64_t* m = t->anc.data() + ((size_t)tr * t->n + a) * 2;
    int c = 0;
    for (int j = 0; j < t->n; ++j)
      if ((m[j >> 6] >> (j & 63)) & 1) row[c++] = j;
    row[c++] = a;
    len[r] = c;
  }
  return TV_OK;
}

// Device mirror of the metadata (masks | depths | parents | offsets | status word) and the two
// pinned staging slots; allocated by the first upload, reused by every later one.
// Upload generations count 1, 2, ... and wrap long before the sign bit (0 = "never").
static int32_t next_gen(tv_tree* t) {
  t->upload_gen = t->upload_gen % 0x3fffffff + 1;
  return t->upload_gen;
}

struct BlobLayout {
  size_t anc_b, i32_b, off_b, total, slot_b;
};
static BlobLayout blob_layout(const tv_tree* t) {
  BlobLayout L;
  const size_t nn = (size_t)t->n_trees * t->n;
  L.anc_b = nn * 2 * sizeof(uint64_t);
  L.i32_b = nn * sizeof(int32_t);
  L.off_b = t->offsets.empty() ? 0 : ((t->offsets.size() * sizeof(int32_t) + 15) & ~(size_t)15);
  const size_t meta_b = L.anc_b + 2 * L.i32_b + L.off_b;
  L.total = ((meta_b + 15) & ~(size_t)15) + 16;                 // + status word
  L.slot_b = (L.i32_b + L.off_b + 255) & ~(size_t)255;          // one staged copy of parents (+ offsets)
  return L;
}
static int ensure_device(tv_tree* t, const BlobLayout& L) {
  int dev = 0;
  TV_CUDA_TRY(cudaGetDevice(&dev));
  if (t->d_blob && (t->device != dev || t->blob_bytes != L.total)) return TV_ERR_BAD_ARG;
  if (t->d_blob) return TV_OK;
  TV_CUDA_TRY(cudaMalloc(&t->d_blob, L.total));
  cudaError_t e = cudaMemset((char*)t->d_blob + L.total - 16, 0, 16);   // status words start at zero
  if (e == cudaSuccess) e = cudaHostAlloc(&t->h_stage, 2 * L.slot_b, cudaHostAllocMapped);
  void* mapped = nullptr;
  if (e == cudaSuccess) e = cudaHostGetDevicePointer(&mapped, t->h_stage, 0);
  for (int i = 0; i < 2 && e == cudaSuccess; ++i)
    e = cudaEventCreateWithFlags(&t->staged[i], cudaEventDisableTiming);
  if (e != cudaSuccess) {
    cudaFree(t->d_blob);
    t->d_blob = nullptr;
    if (t->h_stage) cudaFreeHost(t->h_stage);
    t->h_stage = nullptr;
    tv_set_cuda_error(e);
    return TV_ERR_CUDA;
  }
  t->h_stage_dev = (const int32_t*)mapped;
  t->blob_bytes = L.total;
  t->device = dev;
  char* base = (char*)t->d_blob;
  t->d_anc_w = (uint64_t*)base;
  t->d_depth_w = (int32_t*)(base + L.anc_b);
  t->d_parent_w = (int32_t*)(base + L.anc_b + L.i32_b);
  t->d_anc = t->d_anc_w;
  t->d_depth = t->d_depth_w;
  t->d_parent = t->d_parent_w;
  t->d_status = (int32_t*)(base + L.total - 16);
  if (L.off_b) {
    t->d_offsets_w = (int32_t*)(base + L.anc_b + 2 * L.i32_b);
    t->d_offsets = t->d_offsets_w;
  }
  return TV_OK;
}

TV_API int tv_tree_upload(tv_tree* t, void* stream) {
  if (!t) return TV_ERR_BAD_ARG;
  const BlobLayout L = blob_layout(t);
  int st = ensure_device(t, L);
  if (st != TV_OK) return st;
  cudaStream_t s = (cudaStream_t)stream;
  if (tv_tree_meta_fits_params(t->n_trees, t->n, !t->offsets.empty())) {
    // small tree sets: the parents ride in the launch itself
    st = tv_launch_tree_meta_params(t->parent.data(), t->n_trees, t->n, t->d_anc_w, t->d_depth_w, t->d_parent_w,
                                    t->d_status, t->offsets.empty() ? nullptr : t->offsets.data(),
                                    t->d_offsets_w, s);
    if (st != TV_OK) return st;
    next_gen(t);   // host-built trees cannot break a depth bound: only the generation moves on
    t->uploaded = true;
    t->host_meta_valid = true;
    return TV_OK;
  }
  // The parent arrays go into one of two pinned slots; a small kernel reads the slot over the
  // bus and derives masks and depths on the device (no copy-engine hop in front of the verify
  // launch).  A slot is reused only after the kernel that read it two uploads ago has finished.
  const int slot = t->stage_slot;
  t->stage_slot ^= 1;
  TV_CUDA_TRY(cudaEventSynchronize(t->staged[slot]));
  std::memcpy((char*)t->h_stage + slot * L.slot_b, t->parent.data(), L.i32_b);
  const int32_t* off_mapped = nullptr;
  if (L.off_b) {
    std::memcpy((char*)t->h_stage + slot * L.slot_b + L.i32_b, t->offsets.data(),
                t->offsets.size() * sizeof(int32_t));
    off_mapped = (const int32_t*)((const char*)t->h_stage_dev + slot * L.slot_b + L.i32_b);
  }
  st = tv_launch_tree_meta((const int32_t*)((const char*)t->h_stage_dev + slot * L.slot_b), t->n_trees, t->n,
                           t->d_anc_w, t->d_depth_w, t->d_parent_w, t->d_status, off_mapped, t->d_offsets_w, t->n,
                           next_gen(t), s);
  if (st != TV_OK) return st;
  TV_CUDA_TRY(cudaEventRecord(t->staged[slot], s));
  t->uploaded = true;
  t->host_meta_valid = true;
  return TV_OK;
}

// The same metadata from DEVICE-resident parents and offsets (as tv_budget_select leaves them):
// no host copy, no synchronisation.  The host-side metadata of the handle is then stale.
TV_API int tv_forest_upload_device(tv_tree* t, const int32_t* parent_padded, const int32_t* offsets,
                                   int32_t max_depth_bound, void* stream) {
  if (!t || !parent_padded || !offsets || t->offsets.empty()) return TV_ERR_BAD_ARG;
  if (max_depth_bound < 0 || max_depth_bound >= t->n) return TV_ERR_BAD_ARG;
  if (((uintptr_t)parent_padded | (uintptr_t)offsets) & 3) return TV_ERR_BAD_ARG;
  const BlobLayout L = blob_layout(t);
  int st = ensure_device(t, L);
  if (st != TV_OK) return st;
  st = tv_launch_tree_meta(parent_padded, t->n_trees, t->n, t->d_anc_w, t->d_depth_w, t->d_parent_w, t->d_status,
                           offsets, t->d_offsets_w, max_depth_bound, next_gen(t), (cudaStream_t)stream);
  if (st != TV_OK) return st;
  t->max_depth_all = max_depth_bound;
  t->uploaded = true;
  t->host_meta_valid = false;
  return TV_OK;
}

TV_API int tv_tree_meta_device(tv_tree* t, uint64_t* anc, int32_t* depth, void* stream) {
  if (!t) return TV_ERR_BAD_ARG;
  if (!t->uploaded) return TV_ERR_NOT_UPLOADED;
  const size_t nn = (size_t)t->n_trees * t->n;
  cudaStream_t s = (cudaStream_t)stream;
  if (anc) TV_CUDA_TRY(cudaMemcpyAsync(anc, t->d_anc, nn * 2 * sizeof(uint64_t), cudaMemcpyDeviceToHost, s));
  if (depth) TV_CUDA_TRY(cudaMemcpyAsync(depth, t->d_depth, nn * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  TV_CUDA_TRY(cudaStreamSynchronize(s));
  return TV_OK;
}

TV_API int tv_tree_device_status(tv_tree* t, void* stream) {
  if (!t) return TV_ERR_BAD_ARG;
  if (!t->d_status) return TV_ERR_NOT_UPLOADED;
  int32_t st[2] = {0, 0};
  TV_CUDA_TRY(cudaMemcpyAsync(st, t->d_status, sizeof(st), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  TV_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
  if (st[0] == TV_ERR_CUDA) return TV_ERR_CUDA;   // a kernel refused its shared-memory window
  if (st[0] != 0) return TV_ERR_DEVICE_TIMEOUT;
  if (st[1] != 0 && st[1] == t->upload_gen) return TV_ERR_UNSUPPORTED;   // trees deeper than the stated bound
  return TV_OK;
}

TV_API int tv_tree_free(tv_tree* t) {
  if (!t) return TV_OK;
  if (t->d_blob) cudaFree(t->d_blob);
  if (t->h_stage) cudaFreeHost(t->h_stage);
  for (int i = 0; i < 2; ++i)
    if (t->staged[i]) cudaEventDestroy(t->staged[i]);
  delete t;
  return TV_OK;
}

// ---------------------------------------------------------------------------
// Validation shared by verify and commit.
// ---------------------------------------------------------------------------
static bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

static int check_common(const tv_tree* t, const tv_dims* d) {
  if (!t || !d) return TV_ERR_BAD_ARG;
  if (d->L < 1 || d->B < 1 || d->H < 1 || d->T < 1 || d->dk < 1 || d->dv < 1) return TV_ERR_BAD_ARG;
  if (d->rule != TV_GATED && d->rule != TV_GATED_DELTA) return TV_ERR_BAD_ARG;
  if (d->qkv_dtype != TV_F32 && d->qkv_dtype != TV_BF16) return TV_ERR_BAD_ARG;
  if (d->T > TV_MAX_NODES || d->dk > TV_MAX_DIM || d->dv > TV_MAX_DIM) return TV_ERR_UNSUPPORTED;
  if ((d->dk & 3) || (d->dv & 3)) return TV_ERR_UNSUPPORTED;
  if (d->qkv_dtype == TV_BF16 && ((d->dk & 7) || (d->dv & 7))) return TV_ERR_UNSUPPORTED;
  if (t->n != d->T) return TV_ERR_BAD_ARG;
  if (t->n_trees != 1 && t->n_trees != d->B) return TV_ERR_BAD_ARG;
  if (!t->offsets.empty() && t->n_trees != d->B) return TV_ERR_BAD_ARG;   // a packed forest has one tree per request
  if (d->Hk < 0 || d->Hk > d->H || (d->Hk > 0 && d->H % d->Hk != 0)) return TV_ERR_BAD_ARG;
  if ((int64_t)d->L * d->B * d->H > 0x7fffffffLL) return TV_ERR_UNSUPPORTED;
  if (!t->uploaded) return TV_ERR_NOT_UPLOADED;
  return TV_OK;
}

}  // extern "C"

// Strides of the node-indexed tensors: what the caller gave, or the dense head-major layout
// [L][B][heads][T][d] for a tensor class whose three strides are all zero.
int tv_resolve_layout(const tv_dims* d, bool packed, Layout* out) {
  const int64_t H = d->H, Hk = d->Hk ? d->Hk : d->H, T = d->T;
  const int es = d->qkv_dtype == TV_BF16 ? 2 : 4;
  auto zero = [](const tv_strides& s) { return s.b == 0 && s.h == 0 && s.t == 0; };
  if (packed && !(zero(d->qk) && zero(d->v) && zero(d->gate) && zero(d->out))) return TV_ERR_UNSUPPORTED;
  auto resolve = [&](const tv_strides& s, int64_t heads, int64_t dch, int64_t align, Str3* o) -> int {
    if (zero(s)) {
      o->t = dch;
      o->h = T * dch;
      o->b = heads * T * dch;
      return TV_OK;
    }
    if (s.b < 0 || s.h < 0 || s.t < 0) return TV_ERR_BAD_ARG;
    if ((s.b % align) || (s.h % align) || (s.t % align)) return TV_ERR_BAD_ARG;
    // extents larger than one need a stride that clears a row of d channels
    if ((T > 1 && s.t < dch) || (heads > 1 && s.h < dch) || ((int64_t)d->L * d->B > 1 && s.b < dch)) return TV_ERR_BAD_ARG;
    o->b = s.b; o->h = s.h; o->t = s.t;
    return TV_OK;
  };
  int st = resolve(d->qk, Hk, d->dk, 16 / es, &out->qk);
  if (st == TV_OK) st = resolve(d->v, H, d->dv, 16 / es, &out->v);
  if (st == TV_OK) st = resolve(d->gate, H, 1, 1, &out->gate);
  if (st == TV_OK) st = resolve(d->out, H, d->dv, 4, &out->out);
  return st;
}

extern "C" {

static TreeDev tree_dev(const tv_tree* t) {
  TreeDev td;
  td.anc = t->d_anc;
  td.depth = t->d_depth;
  td.parent = t->d_parent;
  td.n_trees = t->n_trees;
  td.max_depth_all = t->max_depth_all;
  td.offsets = t->d_offsets;
  td.capacity = t->capacity;
  return td;
}

TV_API int tv_tree_verify(const tv_tree* tree, const tv_dims* d, const float* S_pre, const void* q,
                   const void* k, const void* v, const float* alpha, const float* beta, float* O,
                   float* U, void* stream) {
  int st = check_common(tree, d);
  if (st != TV_OK) return st;
  if (!S_pre || !q || !k || !v || !alpha || !O) return TV_ERR_BAD_ARG;
  if (d->rule == TV_GATED_DELTA && !beta) return TV_ERR_BAD_ARG;
  if (!aligned16(S_pre) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(O) ||
      !aligned16(U) || ((uintptr_t)alpha & 3) || ((uintptr_t)beta & 3))
    return TV_ERR_BAD_ARG;
  if (d->impl != TV_IMPL_AUTO && d->impl != TV_IMPL_SIMT && d->impl != TV_IMPL_TC) return TV_ERR_BAD_ARG;
  VerifyArgs a;
  a.tree = tree_dev(tree);
  a.L = d->L; a.B = d->B; a.H = d->H; a.T = d->T; a.dk = d->dk; a.dv = d->dv;
  a.rule = d->rule; a.bf16 = d->qkv_dtype == TV_BF16; a.Hk = d->Hk ? d->Hk : d->H;
  a.S_pre = S_pre; a.q = q; a.k = k; a.v = v; a.alpha = alpha; a.beta = beta; a.O = O; a.U = U;
  st = tv_resolve_layout(d, !tree->offsets.empty(), &a.lay);
  if (st != TV_OK) return st;
  const bool tc_gated = tv_verify_tc_supports(a), tc_delta = tv_verify_tc_delta_supports(a),
             tc_delta128 = tv_verify_tc_delta128_supports(a);
  if (d->impl == TV_IMPL_TC && !tc_gated && !tc_delta && !tc_delta128) return TV_ERR_UNSUPPORTED;
  if (d->impl != TV_IMPL_SIMT) {
    if (tc_gated) return tv_launch_verify_tc(a, tree->d_status, (cudaStream_t)stream);
    if (tc_delta) return tv_launch_verify_tc_delta(a, tree->d_status, (cudaStream_t)stream);
    if (tc_delta128) return tv_launch_verify_tc_delta128(a, tree->d_status, (cudaStream_t)stream);
  }
  return tv_launch_verify_simt(a, (cudaStream_t)stream);
}

// Shared by the two commit entry points: validation of one layer's pointers.
static int check_commit_layer(const tv_dims* d, const float* S_pre, const void* k, const void* v,
                              const float* alpha, const float* beta, const float* U, float* S_new) {
  if (!S_pre || !k || !alpha || !S_new) return TV_ERR_BAD_ARG;
  if (!U && !v) return TV_ERR_BAD_ARG;
  if (d->rule == TV_GATED_DELTA && !U && !beta) return TV_ERR_BAD_ARG;
  if (!aligned16(S_pre) || !aligned16(S_new) || !aligned16(k) || !aligned16(v) || !aligned16(U) ||
      ((uintptr_t)alpha & 3) || ((uintptr_t)beta & 3))
    return TV_ERR_BAD_ARG;
  return TV_OK;
}

static int commit_args(const tv_tree* tree, const tv_dims* d, const int32_t* accepted, bool has_U,
                       bool in_place, CommitArgs* a) {
  a->tree = tree_dev(tree);
  a->L = d->L; a->B = d->B; a->H = d->H; a->T = d->T; a->dk = d->dk; a->dv = d->dv;
  a->rule = d->rule; a->bf16 = d->qkv_dtype == TV_BF16; a->Hk = d->Hk ? d->Hk : d->H;
  a->has_U = has_U; a->in_place = in_place;
  a->accepted = accepted;
  return tv_resolve_layout(d, !tree->offsets.empty(), &a->lay);
}

TV_API int tv_commit_path(const tv_tree* tree, const tv_dims* d, const int32_t* accepted,
                   const float* S_pre, const void* k, const void* v, const float* alpha,
                   const float* beta, const float* U, float* S_new, void* stream) {
  int st = check_common(tree, d);
  if (st != TV_OK) return st;
  if (!accepted || ((uintptr_t)accepted & 3)) return TV_ERR_BAD_ARG;
  st = check_commit_layer(d, S_pre, k, v, alpha, beta, U, S_new);
  if (st != TV_OK) return st;
  const size_t state_elems = (size_t)d->B * d->H * d->dv * d->dk;   // one layer
  if (S_new != S_pre) {
    const size_t bytes = sizeof(float) * (size_t)d->L * state_elems;
    const char* a0 = (const char*)S_pre;
    const char* b0 = (const char*)S_new;
    if (a0 < b0 + bytes && b0 < a0 + bytes) return TV_ERR_BAD_ARG;  // partial overlap
  }
  if (d->rule == TV_GATED_DELTA && !U && d->dk != 64 && d->dk != 128) return TV_ERR_UNSUPPORTED;
  CommitArgs a;
  st = commit_args(tree, d, accepted, U != nullptr, S_new == S_pre, &a);
  if (st != TV_OK) return st;
  // Layers stacked in one allocation: layer l of a node-indexed tensor starts B batch strides
  // (or, in a packed forest, `heads` planes) after layer l-1.
  const size_t es = d->qkv_dtype == TV_BF16 ? 2 : 4;
  size_t k_step, v_step, g_step, u_step;
  if (tree->offsets.empty()) {
    k_step = (size_t)d->B * a.lay.qk.b * es;
    v_step = (size_t)d->B * a.lay.v.b * es;
    g_step = (size_t)d->B * a.lay.gate.b * 4;
    u_step = (size_t)d->B * a.lay.out.b * 4;
  } else {
    const size_t cap = (size_t)tree->capacity;
    k_step = (size_t)a.Hk * cap * d->dk * es;
    v_step = (size_t)d->H * cap * d->dv * es;
    g_step = (size_t)d->H * cap * 4;
    u_step = (size_t)d->H * cap * d->dv * 4;
  }
  // one launch per kCommitMaxLayers layers (one launch in all for the usual 24..64 layers)
  for (int l0 = 0; l0 < d->L; l0 += kCommitMaxLayers) {
    CommitLayers tb = {};
    a.L = d->L - l0 < kCommitMaxLayers ? d->L - l0 : kCommitMaxLayers;
    for (int i = 0; i < a.L; ++i) {
      const size_t l = (size_t)(l0 + i);
      tb.S_pre[i] = S_pre + l * state_elems;
      tb.S_new[i] = S_new + l * state_elems;
      tb.k[i] = (const char*)k + l * k_step;
      tb.v[i] = v ? (const char*)v + l * v_step : nullptr;
      tb.alpha[i] = (const float*)((const char*)alpha + l * g_step);
      tb.beta[i] = beta ? (const float*)((const char*)beta + l * g_step) : nullptr;
      tb.U[i] = U ? (const float*)((const char*)U + l * u_step) : nullptr;
    }
    st = tv_launch_commit(a, tb, (cudaStream_t)stream);
    if (st != TV_OK) return st;
  }
  return TV_OK;
}

TV_API int tv_commit_path_layers(const tv_tree* tree, const tv_dims* d, const int32_t* accepted, int32_t n_layers,
                                 const float* const* S_pre, const void* const* k, const void* const* v,
                                 const float* const* alpha, const float* const* beta, const float* const* U,
                                 float* const* S_new, void* stream) {
  if (!d || n_layers < 1) return TV_ERR_BAD_ARG;
  tv_dims dl = *d;
  dl.L = 1;                         // every table entry is one layer
  int st = check_common(tree, &dl);
  if (st != TV_OK) return st;
  if (!accepted || ((uintptr_t)accepted & 3) || !S_pre || !k || !alpha || !S_new) return TV_ERR_BAD_ARG;
  if (!U && !v) return TV_ERR_BAD_ARG;
  if (d->rule == TV_GATED_DELTA && !U && !beta) return TV_ERR_BAD_ARG;
  if (d->rule == TV_GATED_DELTA && !U && d->dk != 64 && d->dk != 128) return TV_ERR_UNSUPPORTED;
  const size_t bytes = sizeof(float) * (size_t)d->B * d->H * d->dv * d->dk;
  const bool in_place = S_new[0] == S_pre[0];
  for (int l = 0; l < n_layers; ++l) {
    st = check_commit_layer(&dl, S_pre[l], k[l], v ? v[l] : nullptr, alpha[l], beta ? beta[l] : nullptr,
                            U ? U[l] : nullptr, S_new[l]);
    if (st != TV_OK) return st;
    // in place for all layers or for none; no layer's output may overlap any layer's input
    if ((S_new[l] == S_pre[l]) != in_place) return TV_ERR_BAD_ARG;
    for (int m = 0; m < n_layers; ++m) {
      if (in_place && m == l) continue;
      const char* a0 = (const char*)S_pre[m];
      const char* b0 = (const char*)S_new[l];
      if (a0 < b0 + bytes && b0 < a0 + bytes) return TV_ERR_BAD_ARG;
    }
  }
  CommitArgs a;
  st = commit_args(tree, &dl, accepted, U != nullptr, in_place, &a);
  if (st != TV_OK) return st;
  for (int l0 = 0; l0 < n_layers; l0 += kCommitMaxLayers) {
    CommitLayers tb = {};
    a.L = n_layers - l0 < kCommitMaxLayers ? n_layers - l0 : kCommitMaxLayers;
    for (int i = 0; i < a.L; ++i) {
      tb.S_pre[i] = S_pre[l0 + i];
      tb.S_new[i] = S_new[l0 + i];
      tb.k[i] = k[l0 + i];
      tb.v[i] = v ? v[l0 + i] : nullptr;
      tb.alpha[i] = alpha[l0 + i];
      tb.beta[i] = beta ? beta[l0 + i] : nullptr;
      tb.U[i] = U ? U[l0 + i] : nullptr;
    }
    st = tv_launch_commit(a, tb, (cudaStream_t)stream);
    if (st != TV_OK) return st;
  }
  return TV_OK;
}

}  // extern "C"
