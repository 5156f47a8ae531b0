// C ABI of the SamKV library: argument validation, per-request tables, kernel launches.
// Nothing here allocates device memory or synchronises (samkv_poll_status is the one call that does).
#include <stdlib.h>
#include <string.h>

#include <new>

#include <stdio.h>

#include "common.cuh"

using namespace samkv;

namespace {

constexpr size_t kStatusBytes = 256;   // first bytes of the workspace: device status word

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int elem_bytes(const samkv_shape_t& s) { return s.dtype == SAMKV_BF16 ? 2 : 4; }

struct Layout {
  CtxTable ct;
  int nb[SAMKV_MAX_CTX];
  int n_prot[SAMKV_MAX_CTX];
  int n_init_units[SAMKV_MAX_CTX];
  int first_local_unit[SAMKV_MAX_CTX];
  int tail[SAMKV_MAX_CTX];     // tokens in the last unit
  int L_tot, U_tot, max_units;
};

// Validates the shape and derives unit counts and protected ranges.
samkv_status_t make_layout(const samkv_shape_t* s, Layout* lo) {
  if (s == nullptr || s->ctx_offsets == nullptr) return SAMKV_ERR_INVALID_ARG;
  if (s->n_layers < 1 || s->batch < 1 || s->n_q_heads < 1 || s->n_kv_heads < 1) return SAMKV_ERR_INVALID_ARG;
  if (s->n_q_heads % s->n_kv_heads != 0) return SAMKV_ERR_INVALID_ARG;
  if (s->n_q_heads / s->n_kv_heads > 32) return SAMKV_ERR_UNSUPPORTED;   // one warp per query head of a group
  if (s->n_ctx < 1) return SAMKV_ERR_INVALID_ARG;
  if (s->n_ctx > SAMKV_MAX_CTX) return SAMKV_ERR_UNSUPPORTED;
  if (s->head_dim != 64 && s->head_dim != 128) return SAMKV_ERR_UNSUPPORTED;
  if (s->dtype != SAMKV_F32 && s->dtype != SAMKV_BF16) return SAMKV_ERR_UNSUPPORTED;
  const int B = s->block_size;
  if (B < 1 || B > 64 || (B & (B - 1)) != 0) return SAMKV_ERR_UNSUPPORTED;
  if (s->n_init < 0 || s->n_local < 0 || s->n_init % B != 0 || s->n_local % B != 0) return SAMKV_ERR_INVALID_ARG;
  if (s->ctx_offsets[0] != 0) return SAMKV_ERR_INVALID_ARG;
  memset(lo, 0, sizeof(*lo));
  lo->ct.n_ctx = s->n_ctx;
  lo->ct.block_size = B;
  int shift = 0;
  while ((1 << shift) < B) ++shift;
  lo->ct.block_shift = shift;
  lo->max_units = 0;
  for (int c = 0; c < s->n_ctx; ++c) {
    const long long a = s->ctx_offsets[c], b = s->ctx_offsets[c + 1];
    if (b <= a) return SAMKV_ERR_INVALID_ARG;                 // empty or descending context
    const int L_c = (int)(b - a);
    const int nb = (L_c + B - 1) / B;
    if (nb > SAMKV_MAX_UNITS_PER_CTX) return SAMKV_ERR_UNSUPPORTED;
    if (L_c % B != 0 && s->n_local < B) return SAMKV_ERR_INVALID_ARG;   // short tail unit must be protected
    lo->ct.ctx_off[c] = (int)a;
    lo->ct.ctx_off[c + 1] = (int)b;
    lo->ct.unit_off[c + 1] = lo->ct.unit_off[c] + nb;
    lo->nb[c] = nb;
    lo->tail[c] = L_c - (nb - 1) * B;
    // unit m is protected if m*B < n_init, or if its end exceeds L_c - n_local
    int n_init_u = s->n_init / B;
    if (n_init_u > nb) n_init_u = nb;
    int first_local = nb;
    if (s->n_local > 0) {
      const int lim = L_c - s->n_local;                        // units with end > lim are local
      first_local = lim <= 0 ? 0 : lim / B;                    // unit containing token `lim` (end > lim)
    }
    if (first_local < n_init_u) first_local = n_init_u;        // ranges overlap: everything is protected
    lo->n_init_units[c] = n_init_u;
    lo->first_local_unit[c] = first_local;
    lo->n_prot[c] = n_init_u + (nb - first_local);
    if (nb > lo->max_units) lo->max_units = nb;
  }
  lo->L_tot = lo->ct.ctx_off[s->n_ctx];
  lo->U_tot = lo->ct.unit_off[s->n_ctx];
  return SAMKV_OK;
}

// Builds the selection tables for a given k_units; returns the kept-token count in *S.
samkv_status_t make_sel_table(const samkv_shape_t* s, const Layout& lo, const int32_t* k_units, SelTable* st, int* S) {
  if (k_units == nullptr) return SAMKV_ERR_INVALID_ARG;
  memset(st, 0, sizeof(*st));
  for (int c = 0; c < s->n_ctx; ++c) {
    const int k = k_units[c];
    if (k < lo.n_prot[c] || k > lo.nb[c]) return SAMKV_ERR_BUDGET;
    st->sel_off[c + 1] = st->sel_off[c] + k;
    // all units are full except possibly the last one, which is protected (hence kept) when short
    int toks = k * s->block_size;
    if (lo.tail[c] != s->block_size && k > 0) toks -= s->block_size - lo.tail[c];
    st->slot_off[c + 1] = st->slot_off[c] + toks;
    st->n_init_units[c] = lo.n_init_units[c];
    st->first_local_unit[c] = lo.first_local_unit[c];
  }
  *S = st->slot_off[s->n_ctx];
  return SAMKV_OK;
}

size_t qhat_bytes(const samkv_shape_t& s) {
  return round_up((size_t)s.n_layers * s.batch * s.n_ctx * s.n_kv_heads * s.head_dim * sizeof(float), 256);
}

samkv_status_t check_handle(samkv_ctx_impl* h) {
  if (h == nullptr) return SAMKV_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return SAMKV_ERR_CUDA;
  if (dev != h->device) return SAMKV_ERR_CUDA;
  return SAMKV_OK;
}

inline samkv_status_t from_cuda(cudaError_t e) {
#ifdef SAMKV_DEBUG_CHECKS
  if (e != cudaSuccess) fprintf(stderr, "samkv (debug build): CUDA error %d: %s\n", (int)e, cudaGetErrorString(e));
#endif
  return e == cudaSuccess ? SAMKV_OK : SAMKV_ERR_CUDA;
}

}  // namespace

namespace samkv {
// Shape validation + context tables for entry points that live in other files.
samkv_status_t build_ctx_table(const samkv_shape_t* shape, CtxTable* ct) {
  Layout lo;
  samkv_status_t st = make_layout(shape, &lo);
  if (st == SAMKV_OK) *ct = lo.ct;
  return st;
}
}  // namespace samkv

extern "C" {

const char* samkv_status_string(samkv_status_t s) {
  switch (s) {
    case SAMKV_OK: return "ok";
    case SAMKV_ERR_INVALID_ARG: return "invalid argument";
    case SAMKV_ERR_UNSUPPORTED: return "unsupported shape, dtype or size";
    case SAMKV_ERR_WORKSPACE: return "workspace too small";
    case SAMKV_ERR_CAPACITY: return "compact cache capacity too small";
    case SAMKV_ERR_BUDGET: return "k_units outside [protected units, units in context]";
    case SAMKV_ERR_CUDA: return "CUDA runtime error";
    case SAMKV_ERR_DEVICE_CHECK: return "device-side check failed";
  }
  return "unknown status";
}

size_t samkv_workspace_bytes(const samkv_shape_t* shape, int32_t max_q_tokens, int32_t cache_capacity) {
  Layout lo;
  if (make_layout(shape, &lo) != SAMKV_OK || max_q_tokens < 0 || cache_capacity < 0) return 0;
  size_t bytes = kStatusBytes + qhat_bytes(*shape);
  if (max_q_tokens > 0 && cache_capacity > 0) {
    // the plan depends on the SM count; size for the largest split count any device would use
    const size_t out_rows = (size_t)shape->batch * max_q_tokens * shape->n_q_heads;
    const int min_slots = shape->dtype == SAMKV_BF16 ? 256 : 64;
    long long splits = cache_capacity / min_slots;
    if (splits > 64) splits = 64;
    if (splits < 1) splits = 1;
    bytes += round_up(out_rows * (size_t)splits * ((size_t)shape->head_dim * 4 + 8), 256);
  }
  return bytes;
}

samkv_status_t samkv_create(samkv_handle_t* out, int device, void* workspace, size_t workspace_bytes) {
  if (out == nullptr || workspace == nullptr || workspace_bytes < kStatusBytes) return SAMKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return SAMKV_ERR_INVALID_ARG;
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess) return SAMKV_ERR_CUDA;
  if (cur != device) return SAMKV_ERR_CUDA;     // the caller makes `device` current first
  samkv_ctx_impl* h = new (std::nothrow) samkv_ctx_impl;
  if (h == nullptr) return SAMKV_ERR_INVALID_ARG;
  h->device = device;
  h->workspace = static_cast<char*>(workspace);
  h->workspace_bytes = workspace_bytes;
  h->d_status = reinterpret_cast<int*>(workspace);
  h->attn_share_sm = 0;
  if (cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
      cudaDeviceGetAttribute(&h->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess ||
      cudaMemsetAsync(workspace, 0, kStatusBytes, 0) != cudaSuccess) {
    delete h;
    return SAMKV_ERR_CUDA;
  }
  *out = reinterpret_cast<samkv_handle_t>(h);
  return SAMKV_OK;
}

samkv_status_t samkv_attn_share_sm(samkv_handle_t handle, int32_t on) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  h->attn_share_sm = on ? 1 : 0;
  return SAMKV_OK;
}

samkv_status_t samkv_destroy(samkv_handle_t handle) {
  if (handle == nullptr) return SAMKV_ERR_INVALID_ARG;
  delete reinterpret_cast<samkv_ctx_impl*>(handle);
  return SAMKV_OK;
}

samkv_status_t samkv_poll_status(samkv_handle_t handle, void* stream) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int v = 0;
  if (cudaMemcpyAsync(&v, h->d_status, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return SAMKV_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return SAMKV_ERR_CUDA;
  if (v != 0) {
    if (cudaMemsetAsync(h->d_status, 0, sizeof(int), s) != cudaSuccess) return SAMKV_ERR_CUDA;
    return SAMKV_ERR_DEVICE_CHECK;
  }
  return SAMKV_OK;
}

samkv_status_t samkv_layout(const samkv_shape_t* shape, const int32_t* k_units, int32_t* n_protected_out,
                            int32_t* total_units_out, int32_t* kept_tokens_out) {
  Layout lo;
  samkv_status_t st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (n_protected_out != nullptr)
    for (int c = 0; c < shape->n_ctx; ++c) n_protected_out[c] = lo.n_prot[c];
  if (total_units_out != nullptr) *total_units_out = lo.U_tot;
  if (kept_tokens_out != nullptr) {
    SelTable sel;
    int S = 0;
    st = make_sel_table(shape, lo, k_units, &sel, &S);
    if (st != SAMKV_OK) return st;
    *kept_tokens_out = S;
  }
  return SAMKV_OK;
}

samkv_status_t samkv_budget_units(const samkv_shape_t* shape, int32_t budget_bp, int32_t* k_units_out) {
  Layout lo;
  samkv_status_t st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (k_units_out == nullptr || budget_bp < 0 || budget_bp > 10000) return SAMKV_ERR_INVALID_ARG;
  for (int c = 0; c < shape->n_ctx; ++c) {
    long long k = (long long)budget_bp * lo.nb[c] / 10000;
    if (k < lo.n_prot[c]) k = lo.n_prot[c];
    if (k > lo.nb[c]) k = lo.nb[c];
    k_units_out[c] = (int32_t)k;
  }
  return SAMKV_OK;
}

samkv_status_t samkv_score(samkv_handle_t handle, const samkv_shape_t* shape, const void* K, const void* Q, int32_t T_q,
                           const void* Qloc, int32_t T_loc, int32_t use_bias, float* scores_out, float* qhat_out,
                           void* stream) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  Layout lo;
  st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (K == nullptr || Q == nullptr || scores_out == nullptr || T_q < 1) return SAMKV_ERR_INVALID_ARG;
  if (Qloc != nullptr && T_loc < 1) return SAMKV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(Q) || !aligned16(Qloc) || !aligned16(scores_out) || !aligned16(qhat_out))
    return SAMKV_ERR_INVALID_ARG;
  float* qhat = qhat_out;
  if (qhat == nullptr) {
    if (h->workspace_bytes < kStatusBytes + qhat_bytes(*shape)) return SAMKV_ERR_WORKSPACE;
    qhat = reinterpret_cast<float*>(h->workspace + kStatusBytes);
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = launch_qhat(*shape, Q, T_q, Qloc, T_loc, use_bias, qhat, s);
  if (e != cudaSuccess) return from_cuda(e);
  return from_cuda(launch_score(*shape, lo.ct, K, qhat, scores_out, h->d_status, s));
}

samkv_status_t samkv_select(samkv_handle_t handle, const samkv_shape_t* shape, const float* scores,
                            const int32_t* k_units, int32_t* sel_out, void* stream) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  Layout lo;
  st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (scores == nullptr || sel_out == nullptr) return SAMKV_ERR_INVALID_ARG;
  SelTable sel;
  int S = 0;
  st = make_sel_table(shape, lo, k_units, &sel, &S);
  if (st != SAMKV_OK) return st;
  if ((size_t)lo.max_units * 4 + 2048 > (size_t)h->max_smem_optin) return SAMKV_ERR_UNSUPPORTED;
  return from_cuda(launch_select(*shape, lo.ct, sel, scores, k_units, lo.max_units, sel_out, h->d_status,
                                 static_cast<cudaStream_t>(stream)));
}

samkv_status_t samkv_compact(samkv_handle_t handle, const samkv_shape_t* shape, const void* K, const void* V,
                             const int32_t* sel_in, const int32_t* k_units, void* Kc, void* Vc, int32_t cache_capacity,
                             int32_t* cache_len, int32_t* inv_map, void* stream) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  Layout lo;
  st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (K == nullptr || V == nullptr || sel_in == nullptr || Kc == nullptr || Vc == nullptr || cache_len == nullptr)
    return SAMKV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(Kc) || !aligned16(Vc)) return SAMKV_ERR_INVALID_ARG;
  SelTable sel;
  int S = 0;
  st = make_sel_table(shape, lo, k_units, &sel, &S);
  if (st != SAMKV_OK) return st;
  if (cache_capacity < S) return SAMKV_ERR_CAPACITY;
  return from_cuda(launch_compact(*shape, lo.ct, sel, K, V, sel_in, Kc, Vc, cache_capacity, S, cache_len, inv_map,
                                  h->d_status, static_cast<cudaStream_t>(stream)));
}

samkv_status_t samkv_select_compact(samkv_handle_t handle, const samkv_shape_t* shape, const float* scores,
                                    const int32_t* k_units, const void* K, const void* V, int32_t* sel_out, void* Kc,
                                    void* Vc, int32_t cache_capacity, int32_t* cache_len, int32_t* inv_map, void* stream) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  Layout lo;
  st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (scores == nullptr || sel_out == nullptr || K == nullptr || V == nullptr || Kc == nullptr || Vc == nullptr ||
      cache_len == nullptr)
    return SAMKV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(Kc) || !aligned16(Vc)) return SAMKV_ERR_INVALID_ARG;
  SelTable sel;
  int S = 0;
  st = make_sel_table(shape, lo, k_units, &sel, &S);
  if (st != SAMKV_OK) return st;
  if (cache_capacity < S) return SAMKV_ERR_CAPACITY;
  if ((size_t)lo.max_units * 4 + 8192 > (size_t)h->max_smem_optin) return SAMKV_ERR_UNSUPPORTED;
  return from_cuda(launch_select_compact(*shape, lo.ct, sel, scores, lo.max_units, sel_out, K, V, Kc, Vc, cache_capacity, S,
                                         cache_len, inv_map, static_cast<cudaStream_t>(stream)));
}

samkv_status_t samkv_sparsify(samkv_handle_t handle, const samkv_shape_t* shape, const void* K, const void* V,
                              const void* Q, int32_t T_q, const void* Qloc, int32_t T_loc, int32_t use_bias,
                              const int32_t* k_units, float* scores_out, int32_t* sel_out, void* Kc, void* Vc,
                              int32_t cache_capacity, int32_t* cache_len, int32_t* inv_map, void* stream) {
  // every argument is checked before anything is enqueued: the two calls below validate on the host first, and the
  // second one's checks are repeated here so that a refusal leaves nothing half done
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  Layout lo;
  st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (sel_out == nullptr || V == nullptr || Kc == nullptr || Vc == nullptr || cache_len == nullptr) return SAMKV_ERR_INVALID_ARG;
  if (!aligned16(V) || !aligned16(Kc) || !aligned16(Vc)) return SAMKV_ERR_INVALID_ARG;
  SelTable sel;
  int S = 0;
  st = make_sel_table(shape, lo, k_units, &sel, &S);
  if (st != SAMKV_OK) return st;
  if (cache_capacity < S) return SAMKV_ERR_CAPACITY;
  if ((size_t)lo.max_units * 4 + 8192 > (size_t)h->max_smem_optin) return SAMKV_ERR_UNSUPPORTED;
  st = samkv_score(handle, shape, K, Q, T_q, Qloc, T_loc, use_bias, scores_out, nullptr, stream);
  if (st != SAMKV_OK) return st;
  return samkv_select_compact(handle, shape, scores_out, k_units, K, V, sel_out, Kc, Vc, cache_capacity, cache_len, inv_map,
                              stream);
}

samkv_status_t samkv_compact_protected(samkv_handle_t handle, const samkv_shape_t* shape, const void* K, const void* V,
                                       void* Kc, void* Vc, int32_t cache_capacity, int32_t* cache_len,
                                       int32_t* inv_map, void* stream) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  Layout lo;
  st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (K == nullptr || V == nullptr || Kc == nullptr || Vc == nullptr || cache_len == nullptr) return SAMKV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(Kc) || !aligned16(Vc)) return SAMKV_ERR_INVALID_ARG;
  SelTable sel;
  int S = 0;
  st = make_sel_table(shape, lo, lo.n_prot, &sel, &S);
  if (st != SAMKV_OK) return st;
  if (cache_capacity < S) return SAMKV_ERR_CAPACITY;
  return from_cuda(launch_compact(*shape, lo.ct, sel, K, V, nullptr, Kc, Vc, cache_capacity, S, cache_len, inv_map,
                                  h->d_status, static_cast<cudaStream_t>(stream)));
}

samkv_status_t samkv_update(samkv_handle_t handle, const samkv_shape_t* shape, void* Kc, void* Vc,
                            int32_t cache_capacity, const int32_t* inv_map, const int32_t* tok_ids, int32_t R,
                            const void* Knew, const void* Vnew, int32_t mode, void* stream) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  Layout lo;
  st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (R < 0 || cache_capacity < 1) return SAMKV_ERR_INVALID_ARG;
  if (mode != SAMKV_UPDATE_OVERWRITE && mode != SAMKV_UPDATE_FUSION) return SAMKV_ERR_INVALID_ARG;
  if (R == 0) return SAMKV_OK;
  if (Kc == nullptr || Vc == nullptr || inv_map == nullptr || tok_ids == nullptr || Knew == nullptr || Vnew == nullptr)
    return SAMKV_ERR_INVALID_ARG;
  if (!aligned16(Kc) || !aligned16(Vc) || !aligned16(Knew) || !aligned16(Vnew)) return SAMKV_ERR_INVALID_ARG;
  return from_cuda(launch_update(*shape, lo.L_tot, Kc, Vc, cache_capacity, inv_map, tok_ids, R, Knew, Vnew, mode, h->d_status,
                                 static_cast<cudaStream_t>(stream)));
}

samkv_status_t samkv_attn(samkv_handle_t handle, const samkv_shape_t* shape, int32_t layer, void* Kc, void* Vc,
                          int32_t cache_capacity, int32_t* cache_len, const void* Q, int32_t T_q, const void* Kq,
                          const void* Vq, float scale, void* O, float* lse, void* stream) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  Layout lo;
  st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (layer < 0 || layer >= shape->n_layers || T_q < 1 || cache_capacity < 1) return SAMKV_ERR_INVALID_ARG;
  if (Kc == nullptr || Vc == nullptr || cache_len == nullptr || Q == nullptr || O == nullptr)
    return SAMKV_ERR_INVALID_ARG;
  if ((Kq == nullptr) != (Vq == nullptr)) return SAMKV_ERR_INVALID_ARG;
  if (!aligned16(Kc) || !aligned16(Vc) || !aligned16(Q) || !aligned16(O) || !aligned16(Kq) || !aligned16(Vq))
    return SAMKV_ERR_INVALID_ARG;
  if (Kq != nullptr && T_q > cache_capacity) return SAMKV_ERR_CAPACITY;
  const AttnPlan plan = plan_attn(*shape, T_q, cache_capacity, h->sm_count, h->attn_share_sm);
  const size_t ws_off = kStatusBytes + qhat_bytes(*shape);
  if (plan.partial_bytes > 0 && h->workspace_bytes < ws_off + plan.partial_bytes) return SAMKV_ERR_WORKSPACE;
  return from_cuda(launch_attn(*shape, layer, Kc, Vc, cache_capacity, cache_len, Q, T_q, Kq, Vq, scale, O, lse,
                               h->workspace + ws_off, plan, h->d_status, static_cast<cudaStream_t>(stream)));
}

samkv_status_t samkv_attn_layers(samkv_handle_t handle, const samkv_shape_t* shape, int32_t layer0, int32_t n,
                                 void* Kc, void* Vc, int32_t cache_capacity, int32_t* cache_len, const void* Q,
                                 int32_t T_q, const void* Kq, const void* Vq, float scale, void* O, float* lse,
                                 void* stream) {
  if (shape == nullptr || Kc == nullptr || Vc == nullptr || cache_len == nullptr) return SAMKV_ERR_INVALID_ARG;
  if (layer0 < 0 || n < 1 || layer0 > shape->n_layers - n || cache_capacity < 1) return SAMKV_ERR_INVALID_ARG;
  if ((long long)shape->batch * n > 0x7fffffffLL) return SAMKV_ERR_INVALID_ARG;
  // Every tensor is contiguous over the layers, so n layers of Bt requests are one layer of n * Bt requests.
  samkv_shape_t wide = *shape;
  wide.n_layers = 1;
  wide.batch = shape->batch * n;
  const size_t elem = shape->dtype == SAMKV_BF16 ? 2 : 4;
  const size_t layer_bytes = (size_t)shape->batch * shape->n_kv_heads * cache_capacity * shape->head_dim * elem;
  return samkv_attn(handle, &wide, 0, static_cast<char*>(Kc) + layer0 * layer_bytes,
                    static_cast<char*>(Vc) + layer0 * layer_bytes, cache_capacity,
                    cache_len + (size_t)layer0 * shape->batch, Q, T_q, Kq, Vq, scale, O, lse, stream);
}

int32_t samkv_attn_kernel_count(samkv_handle_t handle, const samkv_shape_t* shape, int32_t T_q, int32_t cache_capacity,
                                int32_t appended) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  Layout lo;
  if (h == nullptr || make_layout(shape, &lo) != SAMKV_OK || T_q < 1 || cache_capacity < 1) return 0;
  const AttnPlan plan = plan_attn(*shape, T_q, cache_capacity, h->sm_count, h->attn_share_sm);
  const bool self_merge = shape->dtype == SAMKV_BF16 && attn_merges_in_cluster(plan);
  const bool self_append = shape->dtype == SAMKV_BF16 && shape->head_dim == 128 && plan.rows_per_cta == 128 && !plan.share_sm;
  int n = 1 + ((appended && !self_append) ? 1 : 0);
  if ((plan.n_splits > 1 || appended) && !self_merge) ++n;
  return n;
}

samkv_status_t samkv_topp(samkv_handle_t handle, const samkv_shape_t* shape, const float* scores,
                          const int32_t* star_layers, int32_t n_star, const int32_t* max_units,
                          const int32_t* min_units, float* P_out, void* stream) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  Layout lo;
  st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (scores == nullptr || P_out == nullptr || star_layers == nullptr) return SAMKV_ERR_INVALID_ARG;
  if (n_star < 1 || n_star > SAMKV_MAX_STAR_LAYERS) return SAMKV_ERR_INVALID_ARG;
  for (int i = 0; i < n_star; ++i)
    if (star_layers[i] < 0 || star_layers[i] >= shape->n_layers) return SAMKV_ERR_INVALID_ARG;
  return from_cuda(launch_topp(*shape, lo.ct, lo.n_init_units, lo.first_local_unit, scores, star_layers, n_star,
                               max_units, min_units, P_out, static_cast<cudaStream_t>(stream)));
}

// cand, K, S_u, kept tokens of the cross-context selection; shared by the plan helper and the two calls below
static samkv_status_t cross_plan(const samkv_shape_t* shape, const Layout& lo, const int32_t* cand, int* K, int* S_u,
                                 int* S) {
  long long total = 0, n_prot = 0, deficit = 0;
  for (int c = 0; c < shape->n_ctx; ++c) {
    const int n_mid = lo.nb[c] - lo.n_prot[c];
    if (cand[c] < 0 || cand[c] > n_mid) return SAMKV_ERR_BUDGET;
    total += cand[c];
    n_prot += lo.n_prot[c];
    deficit += shape->block_size - lo.tail[c];
  }
  *K = (int)(total / shape->n_ctx);
  *S_u = (int)(n_prot + *K);
  *S = (int)((long long)*S_u * shape->block_size - deficit);
  return SAMKV_OK;
}

samkv_status_t samkv_topp_plan(const samkv_shape_t* shape, const float* P, int32_t* cand_out, int32_t* K_out,
                               int32_t* S_u_out, int32_t* kept_tokens_out) {
  Layout lo;
  samkv_status_t st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (P == nullptr) return SAMKV_ERR_INVALID_ARG;
  int32_t cand[SAMKV_MAX_CTX];
  for (int c = 0; c < shape->n_ctx; ++c) {
    if (!(P[c] >= 0.0f && P[c] <= 1.0f)) return SAMKV_ERR_INVALID_ARG;       // also refuses NaN
    const int n_mid = lo.nb[c] - lo.n_prot[c];
    int k = (int)((double)P[c] * n_mid + 1e-12);
    if (k > n_mid) k = n_mid;
    cand[c] = k;
    if (cand_out != nullptr) cand_out[c] = k;
  }
  int K = 0, S_u = 0, S = 0;
  st = cross_plan(shape, lo, cand, &K, &S_u, &S);
  if (st != SAMKV_OK) return st;
  if (K_out != nullptr) *K_out = K;
  if (S_u_out != nullptr) *S_u_out = S_u;
  if (kept_tokens_out != nullptr) *kept_tokens_out = S;
  return SAMKV_OK;
}

size_t samkv_select_cross_scratch_bytes(const samkv_shape_t* shape, const int32_t* cand) {
  Layout lo;
  if (make_layout(shape, &lo) != SAMKV_OK) return 0;
  size_t per_slab = 0;                                  // one (key, unit id) pair per retrieved unit
  for (int c = 0; c < shape->n_ctx; ++c) {
    const int n_mid = lo.nb[c] - lo.n_prot[c];
    per_slab += (size_t)(cand == nullptr ? n_mid : (cand[c] < 0 ? 0 : (cand[c] < n_mid ? cand[c] : n_mid)));
  }
  const size_t bytes = (size_t)shape->n_layers * shape->batch * shape->n_kv_heads * per_slab * 8;
  return bytes < 16 ? 16 : bytes;
}

samkv_status_t samkv_select_cross(samkv_handle_t handle, const samkv_shape_t* shape, const float* scores,
                                  const int32_t* cand, void* scratch, size_t scratch_bytes, int32_t* sel_out,
                                  int32_t* counts_out, void* stream) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  Layout lo;
  st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (scores == nullptr || cand == nullptr || sel_out == nullptr) return SAMKV_ERR_INVALID_ARG;
  int K = 0, S_u = 0, S = 0;
  st = cross_plan(shape, lo, cand, &K, &S_u, &S);
  if (st != SAMKV_OK) return st;
  if (scratch == nullptr || !aligned16(scratch)) return SAMKV_ERR_INVALID_ARG;
  if (scratch_bytes < samkv_select_cross_scratch_bytes(shape, cand)) return SAMKV_ERR_WORKSPACE;
  return from_cuda(launch_select_cross(*shape, lo.ct, lo.n_init_units, lo.first_local_unit, scores, cand, K, S_u, scratch,
                                       sel_out, counts_out, h->max_smem_optin, static_cast<cudaStream_t>(stream)));
}

samkv_status_t samkv_compact_units(samkv_handle_t handle, const samkv_shape_t* shape, const void* K, const void* V,
                                   const int32_t* sel_in, int32_t S_u, void* Kc, void* Vc, int32_t cache_capacity,
                                   int32_t* cache_len, int32_t* inv_map, void* stream) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  Layout lo;
  st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (K == nullptr || V == nullptr || sel_in == nullptr || Kc == nullptr || Vc == nullptr || cache_len == nullptr)
    return SAMKV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(Kc) || !aligned16(Vc)) return SAMKV_ERR_INVALID_ARG;
  long long n_prot = 0, deficit = 0;
  for (int c = 0; c < shape->n_ctx; ++c) { n_prot += lo.n_prot[c]; deficit += shape->block_size - lo.tail[c]; }
  if (S_u < n_prot || S_u > lo.U_tot) return SAMKV_ERR_BUDGET;
  const int S = (int)((long long)S_u * shape->block_size - deficit);
  if (cache_capacity < S) return SAMKV_ERR_CAPACITY;
  return from_cuda(launch_compact_units(*shape, lo.ct, lo.n_init_units, lo.first_local_unit, K, V, sel_in, S_u, S, Kc, Vc,
                                        cache_capacity, cache_len, inv_map, h->d_status,
                                        static_cast<cudaStream_t>(stream)));
}

samkv_status_t samkv_block_means(samkv_handle_t handle, const samkv_shape_t* shape, const void* K, void* Kbar,
                                 void* stream) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  Layout lo;
  st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (K == nullptr || Kbar == nullptr || !aligned16(K) || !aligned16(Kbar)) return SAMKV_ERR_INVALID_ARG;
  return from_cuda(launch_block_means(*shape, lo.ct, K, Kbar, h->sm_count, static_cast<cudaStream_t>(stream)));
}

samkv_status_t samkv_score_blocks(samkv_handle_t handle, const samkv_shape_t* shape, const void* Kbar, const void* Q,
                                  int32_t T_q, const void* Qloc, int32_t T_loc, int32_t use_bias, float* scores_out,
                                  float* qhat_out, void* stream) {
  Layout lo;
  samkv_status_t st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  // the representatives form a cache of their own with one "token" per unit
  samkv_shape_t units = *shape;
  units.ctx_offsets = lo.ct.unit_off;
  units.block_size = 1;
  units.n_init = shape->n_init / shape->block_size;
  units.n_local = shape->n_local / shape->block_size;
  return samkv_score(handle, &units, Kbar, Q, T_q, Qloc, T_loc, use_bias, scores_out, qhat_out, stream);
}

samkv_status_t samkv_align(samkv_handle_t handle, const samkv_shape_t* shape, const int32_t* inv_map,
                           const int32_t* tok_ids, int32_t R, uint8_t* flags_out, int32_t* merged_ids,
                           int32_t* merged_len, int32_t* run_ids, int32_t run_capacity, int32_t* run_len, void* stream) {
  samkv_ctx_impl* h = reinterpret_cast<samkv_ctx_impl*>(handle);
  samkv_status_t st = check_handle(h);
  if (st != SAMKV_OK) return st;
  Layout lo;
  st = make_layout(shape, &lo);
  if (st != SAMKV_OK) return st;
  if (inv_map == nullptr || flags_out == nullptr || merged_ids == nullptr || merged_len == nullptr ||
      run_ids == nullptr || run_len == nullptr)
    return SAMKV_ERR_INVALID_ARG;
  if (R < 0 || (R > 0 && tok_ids == nullptr) || run_capacity < 1) return SAMKV_ERR_INVALID_ARG;
  return from_cuda(launch_align(*shape, lo.L_tot, inv_map, tok_ids, R, flags_out, merged_ids, merged_len, run_ids,
                                run_capacity, run_len, h->d_status, static_cast<cudaStream_t>(stream)));
}

}  // extern "C"

#ifdef SAMKV_DEBUG_CHECKS
namespace samkv {
cudaError_t debug_set_score_wait(uint32_t spin_limit, int withhold_first_tile, cudaStream_t stream);
}
// Debug build only (libsamkv_debug.so): samkv_score with the scoring kernel's waits shortened to `spin_limit` polls and
// the copies of every CTA's first tile withheld, so that the bounded wait for that tile runs out.  The kernel records
// the device check, drains and returns; samkv_poll_status then reports SAMKV_ERR_DEVICE_CHECK and later calls work as
// usual.  scores_out is left partly unwritten.
extern "C" samkv_status_t samkv_debug_score_with_lost_copy(samkv_handle_t handle, const samkv_shape_t* shape, const void* K,
                                                           const void* Q, int32_t T_q, const void* Qloc, int32_t T_loc,
                                                           int32_t use_bias, float* scores_out, uint32_t spin_limit,
                                                           void* stream) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (samkv::debug_set_score_wait(spin_limit, 1, s) != cudaSuccess) return SAMKV_ERR_CUDA;
  const samkv_status_t st = samkv_score(handle, shape, K, Q, T_q, Qloc, T_loc, use_bias, scores_out, nullptr, stream);
  if (samkv::debug_set_score_wait(0, 0, s) != cudaSuccess) return SAMKV_ERR_CUDA;
  return st;
}
#endif

