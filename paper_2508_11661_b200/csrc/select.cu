// Per-context selection of SamKV (Sec. 3.2): protected initial/local units are always kept, the
// middle units compete under a fixed budget.  One CTA per (layer, batch, kv head, context):
// the middle scores are turned into order-preserving 32-bit keys held in shared memory, an
// MSB-first radix select (4 passes of 8 bits, two barriers each) finds the k-th largest key, ties at that key are
// broken by index order with a block scan, and the kept ids are emitted already ascending.
#include "common.cuh"

namespace samkv {

constexpr int kSelThreads = 128;

// float -> uint32 with the same ordering; -0 and +0 map to the same key.
__device__ __forceinline__ uint32_t score_key(float x) {
  uint32_t u = __float_as_uint(x);
  if ((u << 1) == 0) u = 0;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exclusive prefix sum over the kSelThreads values held one per thread; also returns the total.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* warp_tot, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  __syncthreads();
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  uint32_t before = 0, tot = 0;
#pragma unroll
  for (int i = 0; i < kSelThreads / 32; ++i) {
    const uint32_t t = warp_tot[i];
    if (i < warp) before += t;
    tot += t;
  }
  *total = tot;
  return before + inc - v;
}

// Selection of one (slab, context): writes the context's segment of the unit list (ascending global unit ids).
// Every thread of the CTA calls it; `keys` holds at least the context's middle units.
__device__ __forceinline__ void select_context(const float* __restrict__ scores, int32_t* __restrict__ sel,
                                               const CtxTable& ct, const SelTable& st, int c, size_t slab, int U_tot,
                                               int S_u, uint32_t* keys, uint32_t* hist, uint32_t* warp_tot,
                                               uint32_t* s_bin, uint32_t* s_remaining, int32_t* list_s = nullptr) {
  const int base = ct.unit_off[c];
  const int nb = ct.unit_off[c + 1] - base;
  const int p0 = st.n_init_units[c];          // middle units are [p0, p1)
  const int p1 = st.first_local_unit[c];
  const int k = st.sel_off[c + 1] - st.sel_off[c];
  const int n_mid = p1 - p0;
  const int k_mid = k - (nb - n_mid);
  int32_t* out = sel + slab * S_u + st.sel_off[c];
  const int tid = threadIdx.x;
  // every list entry also goes to list_s (shared memory) when the caller gathers right after the selection
  auto emit = [&](int j, int unit) {
    out[j] = unit;
    if (list_s != nullptr) list_s[j] = unit;
  };

  // (the protected units are emitted last: list_s may share its memory with the histograms)
  auto emit_protected = [&]() {
    for (int i = tid; i < p0; i += kSelThreads) emit(i, base + i);
    for (int i = p1 + tid; i < nb; i += kSelThreads) emit(k - (nb - p1) + (i - p1), base + i);
  };
  if (k_mid <= 0) { emit_protected(); return; }
  if (k_mid >= n_mid) {
    for (int i = tid; i < n_mid; i += kSelThreads) emit(p0 + i, base + p0 + i);
    emit_protected();
    return;
  }

  const float* sc = scores + slab * U_tot + base + p0;
  for (int i = tid; i < n_mid; i += kSelThreads) keys[i] = score_key(sc[i]);
  for (int i = tid; i < 4 * 256; i += kSelThreads) hist[i] = 0;
  __syncthreads();

  // ---- radix select: the k_mid-th largest key ----
  // One histogram per pass (all zeroed up front) and the bin search done by warp 0 alone with shuffles: two block
  // barriers per pass.  The kernel is bound by barrier latency, not by bytes.
  uint32_t prefix = 0, mask = 0, remaining = (uint32_t)k_mid;
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    uint32_t* h = hist + pass * 256;
    for (int i = tid; i < n_mid; i += kSelThreads) {
      const uint32_t key = keys[i];
      if ((key & mask) == prefix) atomicAdd(&h[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid < 32) {
      // lane L owns bins [8L, 8L + 8); `above` = candidates in higher bins
      uint32_t cnt[8], mine = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { cnt[i] = h[tid * 8 + i]; mine += cnt[i]; }
      uint32_t suffix = mine;                                   // inclusive sum over lanes >= this one
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_down_sync(0xffffffffu, suffix, o);
        if (tid + o < 32) suffix += n;
      }
      uint32_t above = suffix - mine;
#pragma unroll
      for (int i = 7; i >= 0; --i) {
        if (above < remaining && above + cnt[i] >= remaining) {   // exactly one bin of one lane satisfies this
          *s_bin = tid * 8 + i;
          *s_remaining = remaining - above;
        }
        above += cnt[i];
      }
    }
    __syncthreads();
    prefix |= *s_bin << shift;
    mask |= 255u << shift;
    remaining = *s_remaining;
  }
  const uint32_t pivot = prefix;       // k-th largest key
  const uint32_t need_eq = remaining;  // how many keys equal to the pivot are kept (lowest indices first)

  // ---- ordered compaction: contiguous segment per thread, packed (greater, equal) counts ----
  const int per = (n_mid + kSelThreads - 1) / kSelThreads;
  const int a = min(tid * per, n_mid), b = min(a + per, n_mid);
  uint32_t gt = 0, eq = 0;
  for (int i = a; i < b; ++i) {
    const uint32_t key = keys[i];
    gt += key > pivot;
    eq += key == pivot;
  }
  uint32_t total;
  const uint32_t packed = block_exclusive_scan((gt << 16) | eq, warp_tot, &total);
  uint32_t gt_before = packed >> 16, eq_before = packed & 0xffffu;
  for (int i = a; i < b; ++i) {
    const uint32_t key = keys[i];
    if (key > pivot) {
      emit(p0 + gt_before + min(eq_before, need_eq), base + p0 + i);
      ++gt_before;
    } else if (key == pivot) {
      if (eq_before < need_eq) emit(p0 + gt_before + eq_before, base + p0 + i);
      ++eq_before;
    }
  }
  emit_protected();
}

__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, int32_t* __restrict__ sel, const __grid_constant__ CtxTable ct,
              const __grid_constant__ SelTable st, int U_tot, int S_u) {
  extern __shared__ uint32_t keys[];         // [n_mid]
  __shared__ uint32_t hist[4 * 256];         // one histogram per radix pass
  __shared__ uint32_t warp_tot[kSelThreads / 32];
  __shared__ uint32_t s_bin, s_remaining;
  select_context(scores, sel, ct, st, (int)(blockIdx.x % ct.n_ctx), blockIdx.x / ct.n_ctx, U_tot, S_u, keys, hist, warp_tot,
                 &s_bin, &s_remaining);
}

// Selection and compaction of one (slab, context) in one CTA (Sec. 3.2: score -> select -> concatenate in original
// order): the context's unit list is written as by select_kernel, then the same CTA gathers the kept K/V rows of the
// context into the compact cache and fills the inverse map, as compact_kernel does.  The latency-bound selection of
// one CTA overlaps the memory-bound gather of the other CTAs on the SM, and the list never makes a round trip
// through another launch.
template <int kRowBytes>
__global__ void __launch_bounds__(kSelThreads)
select_compact_kernel(const float* __restrict__ scores, int32_t* __restrict__ sel, const char* __restrict__ K,
                      const char* __restrict__ V, char* __restrict__ Kc, char* __restrict__ Vc,
                      int32_t* __restrict__ cache_len, int32_t* __restrict__ inv_map,
                      const __grid_constant__ CtxTable ct, const __grid_constant__ SelTable st, int Hkv, int U_tot, int S_u,
                      int L_tot, int S, int capacity) {
  extern __shared__ uint32_t keys[];
  __shared__ uint32_t hist[4 * 256];
  __shared__ uint32_t warp_tot[kSelThreads / 32];
  __shared__ uint32_t s_bin, s_remaining;
  const int c = (int)(blockIdx.x % ct.n_ctx);
  const size_t slab = blockIdx.x / ct.n_ctx;
  if (c == 0 && threadIdx.x == 0 && (slab % Hkv) == 0) cache_len[slab / Hkv] = S;
  // The context's unit list also stays in shared memory for the gather, in the histograms' memory (dead once the
  // pivot is known), when it fits there.
  int32_t* list_s = (st.sel_off[c + 1] - st.sel_off[c]) <= 4 * 256 ? reinterpret_cast<int32_t*>(hist) : nullptr;
  select_context(scores, sel, ct, st, c, slab, U_tot, S_u, keys, hist, warp_tot, &s_bin, &s_remaining, list_s);
  __syncthreads();                             // the CTA's own list entries are visible to all of its threads

  constexpr int kLanes = kRowBytes / 16;
  constexpr int kRowsPerPass = kSelThreads / kLanes;
  constexpr int kUnroll = 4;
  const int lane = threadIdx.x % kLanes, rsub = threadIdx.x / kLanes;
  const int32_t* list = list_s != nullptr ? list_s : sel + slab * S_u + st.sel_off[c];
  const int slot0 = st.slot_off[c], n_slots = st.slot_off[c + 1] - slot0;
  for (int r0 = 0; r0 < n_slots; r0 += kRowsPerPass * kUnroll) {
    uint4 kv[kUnroll], vv[kUnroll];
    int tok[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int r = r0 + u * kRowsPerPass + rsub;
      tok[u] = -1;
      if (r < n_slots) {
        const int m = list[r >> ct.block_shift] - ct.unit_off[c];
        tok[u] = ct.ctx_off[c] + (m << ct.block_shift) + (r & (ct.block_size - 1));
        const size_t src = (slab * L_tot + tok[u]) * kRowBytes + lane * 16;
        kv[u] = *reinterpret_cast<const uint4*>(K + src);
        vv[u] = ld_stream(V + src);
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      if (tok[u] >= 0) {
        const int slot = slot0 + r0 + u * kRowsPerPass + rsub;
        const size_t dst = (slab * capacity + slot) * kRowBytes + lane * 16;
        *reinterpret_cast<uint4*>(Kc + dst) = kv[u];
        *reinterpret_cast<uint4*>(Vc + dst) = vv[u];
        if (inv_map != nullptr && lane == 0) inv_map[slab * L_tot + tok[u]] = slot;
      }
    }
  }
}

cudaError_t launch_select(const samkv_shape_t& s, const CtxTable& ct, const SelTable& st, const float* scores,
                          const int32_t* k_units_host, int max_units, int32_t* sel, int* d_status,
                          cudaStream_t stream) {
  (void)k_units_host;
  const long long blocks = (long long)s.n_layers * s.batch * s.n_kv_heads * ct.n_ctx;
  if (blocks == 0) return cudaSuccess;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  const size_t smem = (size_t)max_units * sizeof(uint32_t);
  if (smem > 48 * 1024) {
    cudaError_t e = ensure_dynamic_smem<6>(select_kernel, (int)smem);
    if (e != cudaSuccess) return e;
  }
  (void)d_status;
  select_kernel<<<(unsigned)blocks, kSelThreads, smem, stream>>>(scores, sel, ct, st, ct.unit_off[ct.n_ctx],
                                                                st.sel_off[ct.n_ctx]);
  return cudaGetLastError();
}

template <int kRowBytes>
static cudaError_t launch_select_compact_t(const samkv_shape_t& s, const CtxTable& ct, const SelTable& st,
                                           const float* scores, int max_units, int32_t* sel, const void* K, const void* V,
                                           void* Kc, void* Vc, int capacity, int S, int32_t* cache_len, int32_t* inv_map,
                                           cudaStream_t stream) {
  const long long blocks = (long long)s.n_layers * s.batch * s.n_kv_heads * ct.n_ctx;
  if (blocks == 0) return cudaSuccess;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  const size_t smem = (size_t)max_units * sizeof(uint32_t);
  if (smem > 48 * 1024) {
    cudaError_t e = ensure_dynamic_smem<1000 + kRowBytes>(select_compact_kernel<kRowBytes>, (int)smem);
    if (e != cudaSuccess) return e;
  }
  const int L_tot = ct.ctx_off[ct.n_ctx];
  if (inv_map != nullptr) {
    const size_t bytes = (size_t)s.n_layers * s.batch * s.n_kv_heads * L_tot * sizeof(int32_t);
    cudaError_t e = cudaMemsetAsync(inv_map, 0xff, bytes, stream);
    if (e != cudaSuccess) return e;
  }
  select_compact_kernel<kRowBytes><<<(unsigned)blocks, kSelThreads, smem, stream>>>(
      scores, sel, (const char*)K, (const char*)V, (char*)Kc, (char*)Vc, cache_len, inv_map, ct, st, s.n_kv_heads,
      ct.unit_off[ct.n_ctx], st.sel_off[ct.n_ctx], L_tot, S, capacity);
  return cudaGetLastError();
}

cudaError_t launch_select_compact(const samkv_shape_t& s, const CtxTable& ct, const SelTable& st, const float* scores,
                                  int max_units, int32_t* sel, const void* K, const void* V, void* Kc, void* Vc,
                                  int capacity, int S, int32_t* cache_len, int32_t* inv_map, cudaStream_t stream) {
  const int row_bytes = s.head_dim * (s.dtype == SAMKV_BF16 ? 2 : 4);
  switch (row_bytes) {
    case 128: return launch_select_compact_t<128>(s, ct, st, scores, max_units, sel, K, V, Kc, Vc, capacity, S, cache_len, inv_map, stream);
    case 256: return launch_select_compact_t<256>(s, ct, st, scores, max_units, sel, K, V, Kc, Vc, capacity, S, cache_len, inv_map, stream);
    case 512: return launch_select_compact_t<512>(s, ct, st, scores, max_units, sel, K, V, Kc, Vc, capacity, S, cache_len, inv_map, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace samkv
