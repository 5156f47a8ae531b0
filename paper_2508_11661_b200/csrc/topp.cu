// The paper's dynamic selection (Sec. 3.2): Top-P per document from anchor / max / min scores (Eq. 2),
// averaged over the stable layers (Eq. 3), then the cross-context Top-K over the retrieved blocks; and
// the gather for the resulting unit lists, whose per-context counts differ from head to head.
#include <math.h>

#include "common.cuh"

namespace samkv {

constexpr int kTopThreads = 256;       // Top-P and the cross-context stage: few CTAs, many keys each
constexpr int kRetrieveThreads = 128;  // per-document retrieval: many small CTAs, bound by per-CTA latency
constexpr int kTopMaxWarps = kTopThreads / 32;

__device__ __forceinline__ uint32_t order_key(float x) {      // float -> uint32, same ordering, -0 == +0
  uint32_t u = __float_as_uint(x);
  if ((u << 1) == 0) u = 0;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_to_float(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// ---- block-wide helpers (kTopThreads threads) ------------------------------------------------------
struct BlockScratch {
  uint32_t hist[4 * 256];          // one histogram per radix pass
  uint32_t warp_tot[kTopMaxWarps];
  float fred[3][kTopMaxWarps];
  uint32_t bin, remaining;
};

template <int kT>
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, BlockScratch& sc, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  __syncthreads();
  if (lane == 31) sc.warp_tot[warp] = inc;
  __syncthreads();
  uint32_t before = 0, tot = 0;
#pragma unroll
  for (int i = 0; i < kT / 32; ++i) {
    const uint32_t t = sc.warp_tot[i];
    if (i < warp) before += t;
    tot += t;
  }
  *total = tot;
  return before + inc - v;
}

// (sum, max, min) over the block in a fixed order
template <int kT>
__device__ __forceinline__ void block_reduce3(float& s, float& mx, float& mn, BlockScratch& sc) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, o);
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __syncthreads();
  if (lane == 0) { sc.fred[0][warp] = s; sc.fred[1][warp] = mx; sc.fred[2][warp] = mn; }
  __syncthreads();
  s = 0.f; mx = -INFINITY; mn = INFINITY;
  for (int i = 0; i < kT / 32; ++i) {
    s += sc.fred[0][i];
    mx = fmaxf(mx, sc.fred[1][i]);
    mn = fminf(mn, sc.fred[2][i]);
  }
}

// k-th largest of the non-zero keys keys[0..n) (zero marks "not a candidate"); 1 <= k <= number of candidates.
// Returns the pivot key and how many keys equal to it belong to the top k (lowest indices first).
// MSB-first radix select, 4 passes of 8 bits: one histogram per pass (zeroed up front), the bin search by warp 0
// with shuffles, two block barriers per pass.
template <int kT>
__device__ __forceinline__ void block_radix_select(const uint32_t* keys, int n, uint32_t k, BlockScratch& sc,
                                                   uint32_t* pivot, uint32_t* need_eq) {
  const int tid = threadIdx.x;
  for (int i = tid; i < 4 * 256; i += kT) sc.hist[i] = 0;
  __syncthreads();
  uint32_t prefix = 0, mask = 0, remaining = k;
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    uint32_t* h = sc.hist + pass * 256;
    for (int i = tid; i < n; i += kT) {
      const uint32_t key = keys[i];
      if (key != 0 && (key & mask) == prefix) atomicAdd(&h[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid < 32) {
      uint32_t c[8], mine = 0;                                   // lane L owns bins [8L, 8L + 8)
#pragma unroll
      for (int i = 0; i < 8; ++i) { c[i] = h[tid * 8 + i]; mine += c[i]; }
      uint32_t suffix = mine;                                    // inclusive sum over lanes >= this one
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_down_sync(0xffffffffu, suffix, o);
        if (tid + o < 32) suffix += v;
      }
      uint32_t above = suffix - mine;
#pragma unroll
      for (int i = 7; i >= 0; --i) {
        if (above < remaining && above + c[i] >= remaining) { sc.bin = tid * 8 + i; sc.remaining = remaining - above; }
        above += c[i];
      }
    }
    __syncthreads();
    prefix |= sc.bin << shift;
    mask |= 255u << shift;
    remaining = sc.remaining;
  }
  *pivot = prefix;
  *need_eq = remaining;
}

struct StarLayers {
  int n;
  int layer[64];                    // stable layers N* (Eq. 3)
};

struct TopTable {
  int n_init_units[SAMKV_MAX_CTX];
  int first_local_unit[SAMKV_MAX_CTX];
  int cand[SAMKV_MAX_CTX];          // units retrieved per context (cross-context selection)
  int cand_off[SAMKV_MAX_CTX + 1];  // prefix sum of cand: where each context's retrieved units start in the list
  int prot_before[SAMKV_MAX_CTX + 1];  // prefix sum of protected units
  int deficit_before[SAMKV_MAX_CTX + 1];   // tokens missing from short tail units of earlier contexts
};

// ---------------------------------------------------------------------------------------------
// Eq. 2 + Eq. 3.  One CTA per (batch element, context); loops over the stable layers and the KV heads.
//   P[b, c] = mean over (n in N*, h) of  (s_max - s_anc) / (s_max - s_min)  if s_anc in (s_min, s_max] else 0
// s_anc: token-weighted mean of the protected units' scores; s_max / s_min: scores of the caller's max / min
// blocks, or the largest / smallest middle-unit score.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kTopThreads)
topp_kernel(const float* __restrict__ scores, const int32_t* __restrict__ max_units,
            const int32_t* __restrict__ min_units, float* __restrict__ P_out, const __grid_constant__ CtxTable ct,
            const __grid_constant__ TopTable tt, const __grid_constant__ StarLayers star, int Bt, int Hkv, int U_tot) {
  __shared__ BlockScratch sc;
  const int c = blockIdx.x % ct.n_ctx;
  const int b = blockIdx.x / ct.n_ctx;
  const int base = ct.unit_off[c], nb = ct.unit_off[c + 1] - base;
  const int p0 = tt.n_init_units[c], p1 = tt.first_local_unit[c];
  const int L_c = ct.ctx_off[c + 1] - ct.ctx_off[c];
  const int B = ct.block_size;
  float acc = 0.f;
  for (int n = 0; n < star.n; ++n) {
    const int l = star.layer[n];
    for (int h = 0; h < Hkv; ++h) {
      const float* u = scores + (((size_t)l * Bt + b) * Hkv + h) * U_tot + base;
      float anc = 0.f, mx = -INFINITY, mn = INFINITY;
      for (int m = threadIdx.x; m < nb; m += kTopThreads) {
        const float v = u[m];
        if (m < p0 || m >= p1) {
          anc += v * (float)(min((m + 1) * B, L_c) - m * B);
        } else {
          mx = fmaxf(mx, v);
          mn = fminf(mn, v);
        }
      }
      block_reduce3<kTopThreads>(anc, mx, mn, sc);
      if (p1 > p0) {
        const int n_prot_tok = min(p0 * B, L_c) + (L_c - min(p1 * B, L_c));
        const float s_anc = n_prot_tok > 0 ? anc / (float)n_prot_tok : 0.f;
        float s_max = mx, s_min = mn;
        bool ok = true;                                    // a block id outside its context contributes P = 0
        if (max_units != nullptr) {
          const int id = max_units[((size_t)l * Bt + b) * ct.n_ctx + c] - base;
          ok = ok && id >= 0 && id < nb;
          if (ok) s_max = u[id];
        }
        if (min_units != nullptr) {
          const int id = min_units[((size_t)l * Bt + b) * ct.n_ctx + c] - base;
          ok = ok && id >= 0 && id < nb;
          if (ok) s_min = u[id];
        }
        if (ok && s_min < s_anc && s_anc <= s_max) acc += (s_max - s_anc) / (s_max - s_min);
      }
    }
  }
  if (threadIdx.x == 0) P_out[(size_t)b * ct.n_ctx + c] = acc / (float)(star.n * Hkv);
}

// ---------------------------------------------------------------------------------------------
// Cross-context Top-K, stage 1.  One CTA per (layer, batch, kv head, context): retrieve the cand[c] best middle
// units of the context (ties: lower index) and append them, ascending by unit id, to the slab's candidate list
// at cand_off[c]: ckey = order key of the min-max normalised score (never 0), cid = global unit id.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kRetrieveThreads)
retrieve_kernel(const float* __restrict__ scores, uint32_t* __restrict__ ckey, int32_t* __restrict__ cid,
                const __grid_constant__ CtxTable ct, const __grid_constant__ TopTable tt, int U_tot, int C_tot) {
  extern __shared__ uint32_t kc[];                              // [n_mid] order keys of the middle units' scores
  __shared__ BlockScratch sc;
  const int c = blockIdx.x % ct.n_ctx;
  const size_t slab = blockIdx.x / ct.n_ctx;
  const int tid = threadIdx.x;
  const int base = ct.unit_off[c];
  const int p0 = tt.n_init_units[c], p1 = tt.first_local_unit[c];
  const int n_mid = p1 - p0, want = min(tt.cand[c], n_mid);
  if (n_mid <= 0 || want <= 0) return;
  const float* u = scores + slab * U_tot + base + p0;
  float dummy = 0.f, hi = -INFINITY, lo = INFINITY;
  for (int i = tid; i < n_mid; i += kRetrieveThreads) {
    const float v = u[i];
    kc[i] = order_key(v);
    hi = fmaxf(hi, v);
    lo = fminf(lo, v);
  }
  block_reduce3<kRetrieveThreads>(dummy, hi, lo, sc);                             // its barriers also publish kc to the block
  uint32_t pivot = 0, need_eq = 0xffffffffu;                    // want == n_mid: every key is above the pivot
  if (want < n_mid) block_radix_select<kRetrieveThreads>(kc, n_mid, (uint32_t)want, sc, &pivot, &need_eq);
  // ordered pass: keys above the pivot, and the first need_eq keys equal to it, in ascending unit order
  const int per = (n_mid + kRetrieveThreads - 1) / kRetrieveThreads;
  const int a = min(tid * per, n_mid), e = min(a + per, n_mid);
  uint32_t gt = 0, eq = 0;
  for (int i = a; i < e; ++i) {
    gt += (kc[i] > pivot);
    eq += (kc[i] == pivot);
  }
  uint32_t total;
  const uint32_t packed = block_excl_scan<kRetrieveThreads>((gt << 16) | eq, sc, &total);      // both counts < 2^16 (units per context)
  uint32_t gt_before = packed >> 16, eq_before = packed & 0xffffu;
  const float range = hi - lo;
  uint32_t* dkey = ckey + slab * C_tot + tt.cand_off[c];
  int32_t* did = cid + slab * C_tot + tt.cand_off[c];
  for (int i = a; i < e; ++i) {
    const uint32_t key = kc[i];
    int pos = -1;
    if (key > pivot) {
      pos = (int)(gt_before + min(eq_before, need_eq));
      ++gt_before;
    } else if (key == pivot) {
      if (eq_before < need_eq) pos = (int)(gt_before + eq_before);
      ++eq_before;
    }
    if (pos >= 0 && pos < want) {
      const float v = range > 0.f ? (key_to_float(key) - lo) / range : 0.f;
      dkey[pos] = order_key(v);                                 // v >= 0: the key has its top bit set
      did[pos] = base + p0 + i;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Cross-context Top-K, stage 2.  One CTA per (layer, batch, kv head): the K best keys of the slab's candidate list
// (ties: lower unit id = earlier in the list), then the ascending list of protected + chosen units.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kTopThreads)
cross_topk_kernel(const uint32_t* __restrict__ ckey_all, const int32_t* __restrict__ cid_all, int32_t* __restrict__ sel,
                  int32_t* __restrict__ counts, const __grid_constant__ CtxTable ct,
                  const __grid_constant__ TopTable tt, int C_tot, int S_u, int K) {
  __shared__ BlockScratch sc;
  __shared__ int s_chosen[SAMKV_MAX_CTX + 1];                   // chosen units per context, then their prefix sum
  const size_t slab = blockIdx.x;
  const uint32_t* ckey = ckey_all + slab * C_tot;
  const int32_t* cid = cid_all + slab * C_tot;
  int32_t* out = sel + slab * S_u;
  const int tid = threadIdx.x;
  const int D = ct.n_ctx;
  for (int i = tid; i <= SAMKV_MAX_CTX; i += kTopThreads) s_chosen[i] = 0;
  __syncthreads();

  if (K > 0) {
    uint32_t pivot = 0, need_eq = 0xffffffffu;                  // K == C_tot: everything retrieved is kept
    if (K < C_tot) block_radix_select<kTopThreads>(ckey, C_tot, (uint32_t)K, sc, &pivot, &need_eq);
    const int per = (C_tot + kTopThreads - 1) / kTopThreads;
    const int a = min(tid * per, C_tot), e = min(a + per, C_tot);
    uint32_t gt = 0, eq = 0;
    for (int i = a; i < e; ++i) {
      gt += (ckey[i] > pivot);
      eq += (ckey[i] == pivot);
    }
    uint32_t total;
    uint32_t gt_before = block_excl_scan<kTopThreads>(gt, sc, &total);
    uint32_t eq_before = block_excl_scan<kTopThreads>(eq, sc, &total);
    int c = (a < e) ? find_segment(tt.cand_off, D, a) : 0;
    for (int i = a; i < e; ++i) {
      while (i >= tt.cand_off[c + 1]) ++c;
      const uint32_t key = ckey[i];
      int rank = -1;                                            // how many chosen units precede this one
      if (key > pivot) {
        rank = (int)(gt_before + min(eq_before, need_eq));
        ++gt_before;
      } else if (key == pivot) {
        if (eq_before < need_eq) rank = (int)(gt_before + eq_before);
        ++eq_before;
      }
      if (rank >= 0 && rank < K) {
        out[tt.prot_before[c] + tt.n_init_units[c] + rank] = cid[i];
        atomicAdd(&s_chosen[c], 1);
      }
    }
  }
  __syncthreads();
  if (tid == 0) {                                               // exclusive prefix over at most 128 contexts
    int run = 0;
    for (int c = 0; c <= D; ++c) { const int n = s_chosen[c]; s_chosen[c] = run; run += n; }
  }
  __syncthreads();
  const int n_prot_tot = tt.prot_before[D];
  for (int p = tid; p < n_prot_tot; p += kTopThreads) {
    const int c = find_segment(tt.prot_before, D, p);
    const int q = p - tt.prot_before[c];
    if (q < tt.n_init_units[c]) out[p + s_chosen[c]] = ct.unit_off[c] + q;
    else out[p + s_chosen[c + 1]] = ct.unit_off[c] + tt.first_local_unit[c] + (q - tt.n_init_units[c]);
  }
  if (counts != nullptr)
    for (int c = tid; c < D; c += kTopThreads)
      counts[slab * D + c] = tt.prot_before[c + 1] - tt.prot_before[c] + s_chosen[c + 1] - s_chosen[c];
}

// ---------------------------------------------------------------------------------------------
// Gather for a free-form ascending unit list (same length S_u for every slab, any split between contexts).
// Unit at list position p lands at slot p*B - (tokens missing from the short tail units of earlier contexts).
// ---------------------------------------------------------------------------------------------
constexpr int kUnitCopyThreads = 64, kUnitCopyRows = 8;    // small CTAs: they share SMs with attention CTAs

template <int kRowBytes>
__global__ void __launch_bounds__(kUnitCopyThreads)
compact_units_kernel(const char* __restrict__ K, const char* __restrict__ V, const int32_t* __restrict__ sel,
                     char* __restrict__ Kc, char* __restrict__ Vc, int32_t* __restrict__ cache_len,
                     int32_t* __restrict__ inv_map, const __grid_constant__ CtxTable ct,
                     const __grid_constant__ TopTable tt, int Hkv, int L_tot, int S_u, int S, int capacity, int chunks,
                     int* __restrict__ d_status) {
  constexpr int kLanes = kRowBytes / 16;
  constexpr int kRowsPerPass = kUnitCopyThreads / kLanes;
  constexpr int kPasses = kUnitCopyRows / kRowsPerPass;
  const int chunk = blockIdx.x % chunks;
  const size_t slab = blockIdx.x / chunks;
  const int lane = threadIdx.x % kLanes, rsub = threadIdx.x / kLanes;
  if (chunk == 0 && threadIdx.x == 0 && (slab % Hkv) == 0) cache_len[slab / Hkv] = S;
  const int B = ct.block_size;
  // virtual row (list position * B + offset in unit) -> (source token, slot), once per row of the CTA
  __shared__ int s_tok[kUnitCopyRows], s_slot[kUnitCopyRows];
  if (threadIdx.x < kUnitCopyRows) {
    const int v = chunk * kUnitCopyRows + threadIdx.x;
    int t = -1, slot = -1;
    if (v < S_u * B) {
      const int pos = v >> ct.block_shift, j = v & (B - 1);
      const int unit = sel[slab * S_u + pos];
      if (unit < 0 || unit >= ct.unit_off[ct.n_ctx]) {
        atomicMax(d_status, (int)CHECK_SEL_RANGE);
      } else {
        const int c = find_segment(ct.unit_off, ct.n_ctx, unit);
        t = ct.ctx_off[c] + ((unit - ct.unit_off[c]) << ct.block_shift) + j;
        slot = pos * B - tt.deficit_before[c] + j;
        if (t >= ct.ctx_off[c + 1]) {
          t = -1;                                                   // beyond the end of a short tail unit
        } else if (slot < 0 || slot >= S) {
          atomicMax(d_status, (int)CHECK_SEL_RANGE);                // the list is not what samkv_select_cross writes
          t = -1;
        }
      }
    }
    s_tok[threadIdx.x] = t;
    s_slot[threadIdx.x] = slot;
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
      const int slot = s_slot[p * kRowsPerPass + rsub];
      const size_t dst = (slab * capacity + slot) * kRowBytes + lane * 16;
      *reinterpret_cast<uint4*>(Kc + dst) = kv[p];
      *reinterpret_cast<uint4*>(Vc + dst) = vv[p];
      if (inv_map != nullptr && lane == 0) inv_map[slab * L_tot + tok[p]] = slot;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------------
static void fill_top_table(const CtxTable& ct, const int* n_init_units, const int* first_local_unit, const int32_t* cand,
                           TopTable* tt) {
  tt->deficit_before[0] = 0;
  tt->cand_off[0] = 0;
  tt->prot_before[0] = 0;
  for (int c = 0; c < ct.n_ctx; ++c) {
    tt->n_init_units[c] = n_init_units[c];
    tt->first_local_unit[c] = first_local_unit[c];
    tt->cand[c] = cand != nullptr ? cand[c] : 0;
    tt->cand_off[c + 1] = tt->cand_off[c] + tt->cand[c];
    const int nb = ct.unit_off[c + 1] - ct.unit_off[c];
    tt->prot_before[c + 1] = tt->prot_before[c] + n_init_units[c] + (nb - first_local_unit[c]);
    const int L_c = ct.ctx_off[c + 1] - ct.ctx_off[c];
    const int tail = L_c - ((L_c - 1) / ct.block_size) * ct.block_size;
    tt->deficit_before[c + 1] = tt->deficit_before[c] + (ct.block_size - tail);
  }
}

cudaError_t launch_topp(const samkv_shape_t& s, const CtxTable& ct, const int* n_init_units, const int* first_local_unit,
                        const float* scores, const int32_t* star_layers, int n_star, const int32_t* max_units,
                        const int32_t* min_units, float* P_out, cudaStream_t stream) {
  TopTable tt;
  fill_top_table(ct, n_init_units, first_local_unit, nullptr, &tt);
  StarLayers star = {};
  star.n = n_star;
  for (int i = 0; i < n_star; ++i) star.layer[i] = star_layers[i];
  topp_kernel<<<s.batch * ct.n_ctx, kTopThreads, 0, stream>>>(scores, max_units, min_units, P_out, ct, tt, star, s.batch,
                                                             s.n_kv_heads, ct.unit_off[ct.n_ctx]);
  return cudaGetLastError();
}

cudaError_t launch_select_cross(const samkv_shape_t& s, const CtxTable& ct, const int* n_init_units,
                                const int* first_local_unit, const float* scores, const int32_t* cand, int K, int S_u,
                                void* scratch, int32_t* sel, int32_t* counts, int max_smem_optin, cudaStream_t stream) {
  TopTable tt;
  fill_top_table(ct, n_init_units, first_local_unit, cand, &tt);
  const int U_tot = ct.unit_off[ct.n_ctx];
  const int C_tot = tt.cand_off[ct.n_ctx];
  const long long slabs = (long long)s.n_layers * s.batch * s.n_kv_heads;
  if (slabs * ct.n_ctx > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  uint32_t* ckey = static_cast<uint32_t*>(scratch);
  int32_t* cid = reinterpret_cast<int32_t*>(ckey + (size_t)slabs * C_tot);
  if (C_tot > 0) {
    int n_mid_max = 0;
    for (int c = 0; c < ct.n_ctx; ++c) n_mid_max = n_mid_max > first_local_unit[c] - n_init_units[c] ? n_mid_max : first_local_unit[c] - n_init_units[c];
    const size_t smem = (size_t)n_mid_max * sizeof(uint32_t);
    if (smem + 2048 > (size_t)max_smem_optin) return cudaErrorInvalidConfiguration;
    if (smem > 48 * 1024) {
      cudaError_t e = ensure_dynamic_smem<8>(retrieve_kernel, (int)smem);
      if (e != cudaSuccess) return e;
    }
    retrieve_kernel<<<(unsigned)(slabs * ct.n_ctx), kRetrieveThreads, smem, stream>>>(scores, ckey, cid, ct, tt, U_tot, C_tot);
  }
  cross_topk_kernel<<<(unsigned)slabs, kTopThreads, 0, stream>>>(ckey, cid, sel, counts, ct, tt, C_tot, S_u, K);
  return cudaGetLastError();
}

cudaError_t launch_compact_units(const samkv_shape_t& s, const CtxTable& ct, const int* n_init_units,
                                 const int* first_local_unit, const void* K, const void* V, const int32_t* sel, int S_u,
                                 int S, void* Kc, void* Vc, int capacity, int32_t* cache_len, int32_t* inv_map,
                                 int* d_status, cudaStream_t stream) {
  TopTable tt;
  fill_top_table(ct, n_init_units, first_local_unit, nullptr, &tt);
  const long long slabs = (long long)s.n_layers * s.batch * s.n_kv_heads;
  const int L_tot = ct.ctx_off[ct.n_ctx];
  if (inv_map != nullptr) {
    cudaError_t e = cudaMemsetAsync(inv_map, 0xff, (size_t)slabs * L_tot * sizeof(int32_t), stream);
    if (e != cudaSuccess) return e;
  }
  const int rows = S_u * ct.block_size;
  const int chunks = rows > 0 ? (rows + kUnitCopyRows - 1) / kUnitCopyRows : 1;
  const long long blocks = slabs * chunks;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  const int row_bytes = s.head_dim * (s.dtype == SAMKV_BF16 ? 2 : 4);
#define SAMKV_LAUNCH_CU(RB)                                                                                         \
  compact_units_kernel<RB><<<(unsigned)blocks, kUnitCopyThreads, 0, stream>>>((const char*)K, (const char*)V, sel, (char*)Kc,     \
                                                                 (char*)Vc, cache_len, inv_map, ct, tt, s.n_kv_heads, \
                                                                 L_tot, S_u, S, capacity, chunks, d_status)
  switch (row_bytes) {
    case 128: SAMKV_LAUNCH_CU(128); break;
    case 256: SAMKV_LAUNCH_CU(256); break;
    case 512: SAMKV_LAUNCH_CU(512); break;
    default: return cudaErrorInvalidValue;
  }
#undef SAMKV_LAUNCH_CU
  return cudaGetLastError();
}

}  // namespace samkv
