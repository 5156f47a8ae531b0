// Compaction and write-back of SamKV.
//   compact: gather of the kept K/V rows into the compact cache in (context, token) order (Sec. 3.2)
//   update : recomputed rows written back by Overwrite or by Fusion, Eq. 4 (Sec. 3.3)
// Both are pure data movement with 16-byte vectors: kLanes adjacent threads move one row.
#include "common.cuh"

namespace samkv {

constexpr int kCopyThreads = 64;
constexpr int kCompactRowsPerCta = 8;

template <int kRowBytes>
__global__ void __launch_bounds__(kCopyThreads)
compact_kernel(const char* __restrict__ K, const char* __restrict__ V, const int32_t* __restrict__ sel,
               char* __restrict__ Kc, char* __restrict__ Vc, int32_t* __restrict__ cache_len,
               int32_t* __restrict__ inv_map, const __grid_constant__ CtxTable ct, const __grid_constant__ SelTable st,
               int Hkv, int L_tot, int S_u, int S, int capacity, int chunks, int* __restrict__ d_status) {
  constexpr int kLanes = kRowBytes / 16;
  constexpr int kRowsPerPass = kCopyThreads / kLanes;
  constexpr int kPasses = kCompactRowsPerCta / kRowsPerPass;
  static_assert(kPasses >= 1, "tile too small");

  const int chunk = blockIdx.x % chunks;
  const size_t slab = blockIdx.x / chunks;
  const int lane = threadIdx.x % kLanes;
  const int rsub = threadIdx.x / kLanes;

  if (chunk == 0 && threadIdx.x == 0 && (slab % Hkv) == 0) cache_len[slab / Hkv] = S;

  // slot -> source token, once per slot of the CTA (one thread each) instead of once per 16-byte lane: the search
  // over the context table and the dependent read of the unit list leave the copy loop
  __shared__ int s_tok[kCompactRowsPerCta];
  if (threadIdx.x < kCompactRowsPerCta) {
    const int slot = chunk * kCompactRowsPerCta + threadIdx.x;
    int t = -1;
    if (slot < S) {
      const int c = find_segment(st.slot_off, ct.n_ctx, slot);
      const int r = slot - st.slot_off[c];
      const int j = r >> ct.block_shift;
      // without a list (sel == nullptr) the kept units are the protected ones: two contiguous ranges per context
      const int m = sel != nullptr ? sel[slab * S_u + st.sel_off[c] + j] - ct.unit_off[c]
                                   : (j < st.n_init_units[c] ? j : st.first_local_unit[c] + (j - st.n_init_units[c]));
      t = ct.ctx_off[c] + (m << ct.block_shift) + (r & (ct.block_size - 1));
      if (m < 0 || m >= ct.unit_off[c + 1] - ct.unit_off[c] || t >= ct.ctx_off[c + 1]) {
        atomicMax(d_status, (int)CHECK_SEL_RANGE);
        t = -1;
      }
    }
    s_tok[threadIdx.x] = t;
  }
  __syncthreads();

  uint4 kv[kPasses], vv[kPasses];
  int tok[kPasses];
#pragma unroll
  for (int p = 0; p < kPasses; ++p) {
    tok[p] = s_tok[p * kRowsPerPass + rsub];
    if (tok[p] >= 0) {
      const size_t src = (slab * L_tot + tok[p]) * kRowBytes + lane * 16;
      kv[p] = *reinterpret_cast<const uint4*>(K + src);
      vv[p] = ld_stream(V + src);
    }
  }
#pragma unroll
  for (int p = 0; p < kPasses; ++p) {
    if (tok[p] >= 0) {
      const int slot = chunk * kCompactRowsPerCta + p * kRowsPerPass + rsub;
      const size_t dst = (slab * capacity + slot) * kRowBytes + lane * 16;
      *reinterpret_cast<uint4*>(Kc + dst) = kv[p];
      *reinterpret_cast<uint4*>(Vc + dst) = vv[p];
      if (inv_map != nullptr && lane == 0) inv_map[slab * L_tot + tok[p]] = slot;
    }
  }
}

cudaError_t launch_compact(const samkv_shape_t& s, const CtxTable& ct, const SelTable& st, const void* K, const void* V,
                           const int32_t* sel, void* Kc, void* Vc, int capacity, int S, int32_t* cache_len,
                           int32_t* inv_map, int* d_status, cudaStream_t stream) {
  const long long slabs = (long long)s.n_layers * s.batch * s.n_kv_heads;
  const int L_tot = ct.ctx_off[ct.n_ctx];
  if (inv_map != nullptr) {
    cudaError_t e = cudaMemsetAsync(inv_map, 0xff, (size_t)slabs * L_tot * sizeof(int32_t), stream);
    if (e != cudaSuccess) return e;
  }
  const int chunks = (S + kCompactRowsPerCta - 1) / kCompactRowsPerCta;
  const long long blocks = slabs * (chunks > 0 ? chunks : 1);
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  const int row_bytes = s.head_dim * (s.dtype == SAMKV_BF16 ? 2 : 4);
#define SAMKV_LAUNCH_COMPACT(RB)                                                                                   \
  compact_kernel<RB><<<(unsigned)blocks, kCopyThreads, 0, stream>>>(                                                \
      (const char*)K, (const char*)V, sel, (char*)Kc, (char*)Vc, cache_len, inv_map, ct, st, s.n_kv_heads, L_tot,    \
      st.sel_off[ct.n_ctx], S, capacity, chunks > 0 ? chunks : 1, d_status)
  switch (row_bytes) {
    case 128: SAMKV_LAUNCH_COMPACT(128); break;
    case 256: SAMKV_LAUNCH_COMPACT(256); break;
    case 512: SAMKV_LAUNCH_COMPACT(512); break;
    default: return cudaErrorInvalidValue;
  }
#undef SAMKV_LAUNCH_COMPACT
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// update: kLanes threads per (layer, batch, recomputed token, kv head) row.
// ------------------------------------------------------------------------------------------------
template <typename T, int kLanes>
__device__ __forceinline__ uint4 fuse_vec(const uint4& nw, const uint4& od) {
  constexpr int kPerVec = ElemTraits<T>::kPerVec;
  float a[kPerVec], b[kPerVec];
  ElemTraits<T>::unpack(nw, a);
  ElemTraits<T>::unpack(od, b);
  float dot = 0.f, na = 0.f, nb = 0.f;
#pragma unroll
  for (int i = 0; i < kPerVec; ++i) {
    dot = fmaf(a[i], b[i], dot);
    na = fmaf(a[i], a[i], na);
    nb = fmaf(b[i], b[i], nb);
  }
#pragma unroll
  for (int o = kLanes / 2; o > 0; o >>= 1) {
    dot += __shfl_xor_sync(0xffffffffu, dot, o);
    na += __shfl_xor_sync(0xffffffffu, na, o);
    nb += __shfl_xor_sync(0xffffffffu, nb, o);
  }
  const float theta = (na > 0.f && nb > 0.f) ? dot / (sqrtf(na) * sqrtf(nb)) : 1.0f;
  float r[kPerVec];
#pragma unroll
  for (int i = 0; i < kPerVec; ++i) r[i] = fmaf(theta, a[i], (1.0f - theta) * b[i]);
  return ElemTraits<T>::pack(r);
}

// A CTA takes kUpdateRowsPerCta consecutive rows of one (layer, batch element).  The token -> slot look-ups
// (tok_ids, then inv_map: two dependent trips to memory) are done once per row by one thread each and left in
// shared memory; the copy loop then has a single trip per row (new and old rows are fetched together), two rows
// per thread group in flight.
constexpr int kUpdateRowsPerCta = 32;

template <typename T, int kHeadDim>
__global__ void __launch_bounds__(kCopyThreads)
update_kernel(T* __restrict__ Kc, T* __restrict__ Vc, const int32_t* __restrict__ inv_map,
              const int32_t* __restrict__ tok_ids, const T* __restrict__ Knew, const T* __restrict__ Vnew, int Bt,
              int Hkv, int R, int L_tot, int capacity, int mode, long long n_rows, int* __restrict__ d_status) {
  constexpr int kPerVec = ElemTraits<T>::kPerVec;
  constexpr int kLanes = kHeadDim / kPerVec;
  constexpr int kRowsPerPass = kCopyThreads / kLanes;
  constexpr int kPasses = kUpdateRowsPerCta / kRowsPerPass;
  static_assert(kPasses >= 2 && kPasses % 2 == 0 && kUpdateRowsPerCta <= kCopyThreads, "update tile shape");
  const int lane = threadIdx.x % kLanes;
  const int group = threadIdx.x / kLanes;
  // blockIdx.y = l*Bt + b; blockIdx.x walks the R*Hkv rows of that (layer, batch element) in 32-bit arithmetic
  const int lb = blockIdx.y;
  const int rh0 = blockIdx.x * kUpdateRowsPerCta;                                      // first r*Hkv + h of the CTA
  __shared__ int s_slot[kUpdateRowsPerCta];
  if (threadIdx.x < kUpdateRowsPerCta) {
    const int rh = rh0 + threadIdx.x;
    const long long row = (long long)lb * (R * Hkv) + rh;                              // ((l*Bt + b)*R + r)*Hkv + h
    int slot = -1;
    if (rh < R * Hkv && row < n_rows) {
      const int r = rh / Hkv, h = rh - r * Hkv;
      const int l = lb / Bt;
      const int t = tok_ids[(size_t)l * R + r];
      const size_t slab = (size_t)lb * Hkv + h;
      if (t >= 0 && t < L_tot) slot = inv_map[slab * L_tot + t];
      // a token id past the sequence or a slot past the cache is skipped and reported (-1 is the regular "skip")
      if (t >= L_tot || t < -1 || slot >= capacity) {
        atomicMax(d_status, (int)CHECK_SEL_RANGE);
        slot = -1;
      }
    }
    s_slot[threadIdx.x] = slot;
  }
  __syncthreads();
  // Whole kLanes-groups take the same branch, and kLanes divides 32, so shuffles inside fuse_vec are
  // executed by complete groups; inactive groups are masked out without leaving the warp.
#pragma unroll 1
  for (int p = 0; p < kPasses; p += 2) {
    uint4 kn[2], vn[2], ko[2], vo[2];
    size_t dst[2];
    bool active[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int i = (p + u) * kRowsPerPass + group;
      const int rh = rh0 + i;
      const int slot = s_slot[i];
      active[u] = slot >= 0;
      kn[u] = vn[u] = ko[u] = vo[u] = make_uint4(0, 0, 0, 0);
      dst[u] = 0;
      if (active[u]) {
        const int h = rh % Hkv;
        const size_t src = ((size_t)lb * (R * Hkv) + rh) * kHeadDim + lane * kPerVec;
        dst[u] = (((size_t)lb * Hkv + h) * capacity + slot) * kHeadDim + lane * kPerVec;
        kn[u] = ld_stream(Knew + src);
        vn[u] = ld_stream(Vnew + src);
        if (mode == SAMKV_UPDATE_FUSION) {
          ko[u] = *reinterpret_cast<const uint4*>(Kc + dst[u]);
          vo[u] = *reinterpret_cast<const uint4*>(Vc + dst[u]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      if (mode == SAMKV_UPDATE_FUSION) {
        kn[u] = fuse_vec<T, kLanes>(kn[u], ko[u]);
        vn[u] = fuse_vec<T, kLanes>(vn[u], vo[u]);
      }
      if (active[u]) {
        *reinterpret_cast<uint4*>(Kc + dst[u]) = kn[u];
        *reinterpret_cast<uint4*>(Vc + dst[u]) = vn[u];
      }
    }
  }
}

cudaError_t launch_update(const samkv_shape_t& s, int L_tot, void* Kc, void* Vc, int capacity, const int32_t* inv_map,
                          const int32_t* tok_ids, int R, const void* Knew, const void* Vnew, int mode, int* d_status,
                          cudaStream_t stream) {
  const long long n_rows = (long long)s.n_layers * s.batch * R * s.n_kv_heads;
  if (n_rows == 0) return cudaSuccess;
#define SAMKV_LAUNCH_UPDATE(T, HD)                                                                                 \
  do {                                                                                                             \
    constexpr int rows_per_cta = kUpdateRowsPerCta;                                                                \
    const long long per_lb = ((long long)R * s.n_kv_heads + rows_per_cta - 1) / rows_per_cta;                      \
    const long long n_lb = (long long)s.n_layers * s.batch;                                                        \
    if (per_lb > 0x7fffffffLL || n_lb > 65535) return cudaErrorInvalidConfiguration;                               \
    update_kernel<T, HD><<<dim3((unsigned)per_lb, (unsigned)n_lb), kCopyThreads, 0, stream>>>((T*)Kc, (T*)Vc, inv_map, tok_ids, \
                                                                       (const T*)Knew, (const T*)Vnew, s.batch,    \
                                                                       s.n_kv_heads, R, L_tot, capacity, mode,     \
                                                                       n_rows, d_status);                          \
  } while (0)
  if (s.dtype == SAMKV_BF16) {
    if (s.head_dim == 128) SAMKV_LAUNCH_UPDATE(__nv_bfloat16, 128); else SAMKV_LAUNCH_UPDATE(__nv_bfloat16, 64);
  } else {
    if (s.head_dim == 128) SAMKV_LAUNCH_UPDATE(float, 128); else SAMKV_LAUNCH_UPDATE(float, 64);
  }
#undef SAMKV_LAUNCH_UPDATE
  return cudaGetLastError();
}

}  // namespace samkv
