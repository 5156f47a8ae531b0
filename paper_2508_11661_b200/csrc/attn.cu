// Attention of a query chunk over the compact multi-context cache (Sec. 3.3: the incremental
// prefill of the user query over the new sparse cache, and the decode steps that follow).
//
// This file holds what every attention path shares — the split-KV plan, the append of the chunk's
// own K/V rows, the merge of split partials — and the fp32 FMA kernel used for fp32 caches
// (tensor cores would round fp32 operands; the fp32 path keeps full fp32 products).
//
// Packed query rows: row r of a (batch, kv head) pair is (token t = r / G, group member g = r % G),
// so the G query heads that share a KV head are adjacent and the causal limit depends on r / G only.
#include <math.h>

#include "common.cuh"

namespace samkv {

constexpr int kSimtWarps = 4;
constexpr float kNegInf = -INFINITY;

cudaError_t launch_attn_mma(const samkv_shape_t& s, int layer, const void* Kc, const void* Vc, int capacity,
                            const int32_t* cache_len, const void* Q, int T_q, int appended, float scale, void* O,
                            float* lse, float* part_o, float2* part_ml, const AttnPlan& plan, cudaStream_t stream);
cudaError_t launch_attn_tc2(const samkv_shape_t& s, const void* Kc, const void* Vc, int capacity,
                            const int32_t* cache_len, const void* Q, int T_q, int appended, float scale, void* O,
                            float* lse, float* part_o, float2* part_ml, const AttnPlan& plan, int* d_status,
                            cudaStream_t stream);
cudaError_t launch_attn_tc3(const samkv_shape_t& s, const void* Kc, const void* Vc, int capacity, int32_t* cache_len,
                            const void* Q, int T_q, int appended, float scale, void* O, float* lse, float* part_o,
                            float2* part_ml, const AttnPlan& plan, int* d_status, cudaStream_t stream);
cudaError_t launch_attn_tc4(const samkv_shape_t& s, void* Kc, void* Vc, int capacity, int32_t* cache_len,
                            const void* Q, int T_q, const void* Kq, const void* Vq, float scale, void* O, float* lse,
                            float* part_o, float2* part_ml, const AttnPlan& plan, int* d_status, cudaStream_t stream);

// ---------------------------------------------------------------------------------------------
// Plan: how many packed rows a CTA takes and into how many KV splits a (batch, kv head) is cut.
// The host does not know cache_len (it lives on the device), so splits are sized from capacity.
// ---------------------------------------------------------------------------------------------
// Best split count for one kernel shape: least (waves x time per CTA), where a CTA costs `tile_cost` per KV tile
// plus `fixed_cost` for its prologue and epilogue (any common unit).  A grid that spills a few CTAs into one more
// wave costs a whole wave.
static long long best_split(long long base_ctas, long long tiles, long long slots, long long max_splits,
                            long long tile_cost, long long fixed_cost, long long* cost_out,
                            long long fixed_cost_3plus = -1, long long fixed_cost_2 = -1) {
  long long best_n = 1, best_cost = -1;
  for (long long n = 1; n <= max_splits; ++n) {
    const long long tps = (tiles + n - 1) / n;
    const long long waves = (base_ctas * n + slots - 1) / slots;
    // (a kernel that merges one or two splits itself pays more once partial results go through global memory)
    const long long fixed = (n >= 3 && fixed_cost_3plus >= 0) ? fixed_cost_3plus
                            : (n == 2 && fixed_cost_2 >= 0)     ? fixed_cost_2 : fixed_cost;
    const long long cost = waves * (tps * tile_cost + fixed);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_n = n; }
  }
  *cost_out = best_cost;
  return best_n;
}

AttnPlan plan_attn(const samkv_shape_t& s, int T_q, int capacity, int sm_count, int share_sm) {
  AttnPlan p;
  p.share_sm = 0;
  const int G = s.n_q_heads / s.n_kv_heads;
  const int rows = T_q * G;
  const long long bh = (long long)s.batch * s.n_kv_heads;
  const long long min_slots = s.dtype == SAMKV_BF16 ? 256 : 64;
  long long max_splits = capacity / min_slots;
  if (max_splits > 64) max_splits = 64;
  if (max_splits < 1) max_splits = 1;
  long long cost = 0;
  if (s.dtype == SAMKV_BF16 && rows >= 128 && s.head_dim == 128) {
    // The two tcgen05 kernels, one CTA per SM, 128-slot tiles.  Measured on B200 (cycles): 256 rows per CTA
    // (two query tiles share every K/V tile, which halves the L2 traffic) ~4070 per tile + ~35000 per CTA;
    // 128 rows per CTA (two groups of tiles taking turns) ~2150 per tile + ~8000 per CTA, ~25000 when two splits
    // merge inside a cluster (the exchange, the partner's imbalance, and clusters that wait for two free SMs once the
    // grid spans several waves), ~30000 with three or more splits, which go through global memory.  The second
    // kernel wins everywhere except on very long KV ranges.
    const long long tiles = (capacity + 127) / 128;
    long long cost256 = 0, cost128 = 0;
    const long long n256 = best_split(bh * ((rows + 255) / 256), tiles, sm_count, max_splits, 4070, 35000, &cost256);
    const long long n128 = best_split(bh * ((rows + 127) / 128), tiles, sm_count, max_splits, 2150, 8000, &cost128, 30000, 25000);
    const bool use128 = cost128 <= cost256;
    p.rows_per_cta = use128 ? 128 : 256;
    p.n_splits = (int)(use128 ? n128 : n256);
    if (share_sm && use128) {
      // The caller runs copy kernels on other streams next to attention: the 128-row kernel with one double-buffered
      // score tile (~2760 per tile + ~9000 per CTA) is slower alone but leaves them room on every SM.
      long long cost_share = 0;
      p.n_splits = (int)best_split(bh * ((rows + 127) / 128), tiles, sm_count, max_splits, 2760, 9000, &cost_share, 22000);
      p.share_sm = 1;
    }
  } else if (s.dtype == SAMKV_BF16) {
    // mma.sync kernel with 64 or 16 rows per CTA, 64-slot tiles; the fixed part is taken as 3 tiles
    p.rows_per_cta = rows > 16 ? 64 : 16;
    const long long ctas_per_sm = rows > 16 ? 2 : 3;          // shared memory / registers of the kernel
    p.n_splits = (int)best_split(bh * ((rows + p.rows_per_cta - 1) / p.rows_per_cta), (capacity + 63) / 64,
                                 sm_count * ctas_per_sm, max_splits, 1, 3, &cost);
  } else {
    p.rows_per_cta = kSimtWarps;
    p.n_splits = (int)best_split(bh * ((rows + kSimtWarps - 1) / kSimtWarps), (capacity + 63) / 64,
                                 (long long)sm_count * 8, max_splits, 1, 3, &cost);
  }
  const size_t out_rows = (size_t)s.batch * T_q * s.n_q_heads;
  p.partial_bytes = p.n_splits > 1 ? out_rows * p.n_splits * ((size_t)s.head_dim * 4 + 8) : 0;
  return p;
}

// ---------------------------------------------------------------------------------------------
// Append: Kc[layer, b, h, cache_len[b] + t, :] = Kq[b, t, h, :] (same for V).  cache_len is not changed
// here; the finalize kernel adds T_q after attention has read it.
// ---------------------------------------------------------------------------------------------
__global__ void append_kernel(char* __restrict__ Kc, char* __restrict__ Vc, const int32_t* __restrict__ cache_len,
                              const char* __restrict__ Kq, const char* __restrict__ Vq, int Hkv, int T_q, int capacity,
                              int row_bytes, long long n_threads, int* __restrict__ d_status) {
  pdl_launch_dependents();      // the attention kernel may set itself up while the chunk is being appended
  pdl_wait();                   // the kernel before this one may be the previous call's attention: it bumps cache_len
  const int lanes = row_bytes / 16;
  const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= n_threads) return;
  const long long row = gid / lanes;                // (b * T_q + t) * Hkv + h
  const int lane = (int)(gid % lanes);
  const int h = (int)(row % Hkv);
  const long long bt = row / Hkv;
  const int t = (int)(bt % T_q);
  const long long b = bt / T_q;
  const int len = cache_len[b];
  if (len < 0 || len + T_q > capacity) {
    if (lane == 0 && t == 0 && h == 0) atomicMax(d_status, (int)CHECK_APPEND_CAPACITY);
    return;
  }
  const size_t src = (size_t)row * row_bytes + lane * 16;
  const size_t dst = (((size_t)b * Hkv + h) * capacity + len + t) * row_bytes + lane * 16;
  *reinterpret_cast<uint4*>(Kc + dst) = *reinterpret_cast<const uint4*>(Kq + src);
  *reinterpret_cast<uint4*>(Vc + dst) = *reinterpret_cast<const uint4*>(Vq + src);
}

// ---------------------------------------------------------------------------------------------
// fp32-FMA attention.  One warp per packed query row; lane e owns kEpl consecutive elements of the
// head dimension.  Works for fp32 and bf16 caches; selected for fp32.
// ---------------------------------------------------------------------------------------------
template <typename T, int kEpl>
__device__ __forceinline__ void load_elems(const T* p, float* f);
template <>
__device__ __forceinline__ void load_elems<float, 4>(const float* p, float* f) {
  const float4 v = *reinterpret_cast<const float4*>(p);
  f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
template <>
__device__ __forceinline__ void load_elems<float, 2>(const float* p, float* f) {
  const float2 v = *reinterpret_cast<const float2*>(p);
  f[0] = v.x; f[1] = v.y;
}
template <>
__device__ __forceinline__ void load_elems<__nv_bfloat16, 4>(const __nv_bfloat16* p, float* f) {
  const uint2 v = *reinterpret_cast<const uint2*>(p);
  f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
}
template <>
__device__ __forceinline__ void load_elems<__nv_bfloat16, 2>(const __nv_bfloat16* p, float* f) {
  const uint32_t v = *reinterpret_cast<const uint32_t*>(p);
  f[0] = bf16_lo(v); f[1] = bf16_hi(v);
}
template <typename T>
__device__ __forceinline__ void store_elem(T* p, float v);
template <>
__device__ __forceinline__ void store_elem<float>(float* p, float v) { *p = v; }
template <>
__device__ __forceinline__ void store_elem<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

template <typename T, int kHeadDim>
__global__ void __launch_bounds__(kSimtWarps * 32)
attn_simt_kernel(const T* __restrict__ Kc, const T* __restrict__ Vc, const int32_t* __restrict__ cache_len,
                 const T* __restrict__ Q, T* __restrict__ O, float* __restrict__ lse, float* __restrict__ part_o,
                 float2* __restrict__ part_ml, int Hq, int Hkv, int T_q, int capacity, int appended, float scale,
                 int n_splits, int row_tiles) {
  constexpr int kEpl = kHeadDim / 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = Hq / Hkv;
  const int split = blockIdx.x % n_splits;
  const int tile = (blockIdx.x / n_splits) % row_tiles;
  const int bh = blockIdx.x / (n_splits * row_tiles);
  const int h = bh % Hkv, b = bh / Hkv;
  const int r = tile * kSimtWarps + warp;
  if (r >= T_q * G) return;
  const int t = r / G, hq = h * G + (r % G);

  int len = cache_len[b];
  len = max(0, min(len, capacity));
  const int n_app = (appended && len + T_q <= capacity) ? T_q : 0;
  const int total = len + n_app;
  const int visible = len + (n_app ? t + 1 : 0);
  // split ranges are cut in multiples of 64 slots of the whole (cache + chunk) range
  const int per = ((total + n_splits - 1) / n_splits + 63) & ~63;
  const int j0 = split * per;
  const int j1 = min(min(j0 + per, total), visible);

  float q[kEpl];
  const size_t orow = ((size_t)b * T_q + t) * Hq + hq;
  load_elems<T, kEpl>(Q + orow * kHeadDim + lane * kEpl, q);
  const T* kbase = Kc + ((size_t)bh * capacity) * kHeadDim + lane * kEpl;
  const T* vbase = Vc + ((size_t)bh * capacity) * kHeadDim + lane * kEpl;

  float m = kNegInf, l = 0.f, acc[kEpl];
#pragma unroll
  for (int i = 0; i < kEpl; ++i) acc[i] = 0.f;

  for (int j = j0; j < j1; ++j) {
    float kf[kEpl], vf[kEpl];
    load_elems<T, kEpl>(kbase + (size_t)j * kHeadDim, kf);
    load_elems<T, kEpl>(vbase + (size_t)j * kHeadDim, vf);
    float dot = 0.f;
#pragma unroll
    for (int i = 0; i < kEpl; ++i) dot = fmaf(q[i], kf[i], dot);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    const float sc = dot * scale;
    const float m_new = fmaxf(m, sc);
    const float corr = expf(m - m_new);      // exp(-inf) = 0 on the first slot
    const float p = expf(sc - m_new);
    l = l * corr + p;
#pragma unroll
    for (int i = 0; i < kEpl; ++i) acc[i] = fmaf(p, vf[i], acc[i] * corr);
    m = m_new;
  }

  if (n_splits == 1) {
    const float inv = l > 0.f ? 1.0f / l : 0.f;
#pragma unroll
    for (int i = 0; i < kEpl; ++i) store_elem<T>(O + orow * kHeadDim + lane * kEpl + i, acc[i] * inv);
    if (lse != nullptr && lane == 0) lse[((size_t)b * Hq + hq) * T_q + t] = l > 0.f ? m + logf(l) : kNegInf;
  } else {
    float* po = part_o + (orow * n_splits + split) * kHeadDim + lane * kEpl;
#pragma unroll
    for (int i = 0; i < kEpl; ++i) po[i] = acc[i];
    if (lane == 0) part_ml[orow * n_splits + split] = make_float2(m, l);
  }
}

// ---------------------------------------------------------------------------------------------
// Finalize: merge split partials (O_s, m_s, l_s) -> O, lse; then cache_len += T_q if a chunk was appended.
// One warp per output row (b, t, hq).
// ---------------------------------------------------------------------------------------------
template <typename T, int kHeadDim>
__global__ void __launch_bounds__(128)
attn_finalize_kernel(const float* __restrict__ part_o, const float2* __restrict__ part_ml, T* __restrict__ O,
                     float* __restrict__ lse, int32_t* __restrict__ cache_len, int Bt, int Hq, int T_q, int capacity,
                     int appended, int n_splits, long long n_rows) {
  constexpr int kEpl = kHeadDim / 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * 4 + warp;
  pdl_wait();                   // the attention kernel's partials and its reads of cache_len are complete
  if (n_splits > 1 && row < n_rows) {
    // lane s holds (m, l) of split s (and of split s + 32): one round trip for all of them, then the maximum,
    // the weights and the denominator by shuffles; the partial rows are then fetched four splits at a time.
    // Sums run over the splits in ascending order, as a plain loop would.
    const float2* ml_row = part_ml + row * n_splits;
    const float2 ml0 = lane < n_splits ? ml_row[lane] : make_float2(kNegInf, 0.f);
    const float2 ml1 = lane + 32 < n_splits ? ml_row[lane + 32] : make_float2(kNegInf, 0.f);
    float M = fmaxf(ml0.x, ml1.x);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    const float w0 = ml0.y > 0.f ? expf(ml0.x - M) : 0.f;      // a split that saw no visible slot weighs nothing
    const float w1 = ml1.y > 0.f ? expf(ml1.x - M) : 0.f;
    float L = 0.f, acc[kEpl];
#pragma unroll
    for (int i = 0; i < kEpl; ++i) acc[i] = 0.f;
    const float* po_row = part_o + row * n_splits * kHeadDim + lane * kEpl;
    for (int s0 = 0; s0 < n_splits; s0 += 4) {
      float po[4][kEpl], w[4], lw[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int s = s0 + u;
        const float ws = __shfl_sync(0xffffffffu, s < 32 ? w0 : w1, s & 31);
        const float ls = __shfl_sync(0xffffffffu, s < 32 ? ml0.y : ml1.y, s & 31);
        w[u] = s < n_splits ? ws : 0.f;
        lw[u] = s < n_splits ? ls * ws : 0.f;
        if (s < n_splits) {
          if constexpr (kEpl == 4) {
            const float4 v = *reinterpret_cast<const float4*>(po_row + (size_t)s * kHeadDim);
            po[u][0] = v.x; po[u][1] = v.y; po[u][2] = v.z; po[u][3] = v.w;
          } else {
            const float2 v = *reinterpret_cast<const float2*>(po_row + (size_t)s * kHeadDim);
            po[u][0] = v.x; po[u][1] = v.y;
          }
        } else {
#pragma unroll
          for (int i = 0; i < kEpl; ++i) po[u][i] = 0.f;
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (w[u] > 0.f) {                                       // skipped splits may hold stale numbers, even NaN
          L += lw[u];
#pragma unroll
          for (int i = 0; i < kEpl; ++i) acc[i] = fmaf(w[u], po[u][i], acc[i]);
        }
      }
    }
    const float inv = L > 0.f ? 1.0f / L : 0.f;
    if constexpr (sizeof(T) == 2 && kEpl == 4) {
      uint2 v;
      v.x = ElemTraits<__nv_bfloat16>::pack2(acc[0] * inv, acc[1] * inv);
      v.y = ElemTraits<__nv_bfloat16>::pack2(acc[2] * inv, acc[3] * inv);
      *reinterpret_cast<uint2*>(O + row * kHeadDim + lane * kEpl) = v;
    } else {
#pragma unroll
      for (int i = 0; i < kEpl; ++i) store_elem<T>(O + row * kHeadDim + lane * kEpl + i, acc[i] * inv);
    }
    if (lse != nullptr && lane == 0) {
      const int hq = (int)(row % Hq);
      const long long bt = row / Hq;
      const int t = (int)(bt % T_q);
      const long long b = bt / T_q;
      lse[((size_t)b * Hq + hq) * T_q + t] = L > 0.f ? M + logf(L) : kNegInf;
    }
  }
  if (appended && blockIdx.x == 0 && threadIdx.x < Bt) {
    // every attention CTA of this call has finished reading cache_len (stream order)
    for (int b = threadIdx.x; b < Bt; b += blockDim.x) {
      const int len = cache_len[b];
      if (len >= 0 && len + T_q <= capacity) cache_len[b] = len + T_q;
    }
  }
}

template <typename T, int kHeadDim>
static cudaError_t launch_attn_t(const samkv_shape_t& s, int layer, void* Kc, void* Vc, int capacity,
                                 int32_t* cache_len, const void* Q, int T_q, const void* Kq, const void* Vq,
                                 float scale, void* O, float* lse, void* partial_ws, const AttnPlan& plan,
                                 int* d_status, cudaStream_t stream) {
  const int Bt = s.batch, Hq = s.n_q_heads, Hkv = s.n_kv_heads;
  const size_t slab_elems = (size_t)Bt * Hkv * capacity * kHeadDim;
  T* Kl = (T*)Kc + (size_t)layer * slab_elems;
  T* Vl = (T*)Vc + (size_t)layer * slab_elems;
  int32_t* len_l = cache_len + (size_t)layer * Bt;
  const int appended = Kq != nullptr;
  const size_t out_rows = (size_t)Bt * T_q * Hq;
  float* part_o = (float*)partial_ws;
  float2* part_ml = (float2*)(part_o + out_rows * plan.n_splits * kHeadDim);

  // the 128-row tensor-memory kernel writes the chunk's rows into the cache itself
  const bool self_append = sizeof(T) == 2 && kHeadDim == 128 && plan.rows_per_cta == 128 && !plan.share_sm;
  if (appended && !self_append) {
    const int row_bytes = kHeadDim * (int)sizeof(T);
    const long long threads = (long long)Bt * T_q * Hkv * (row_bytes / 16);
    // launched as a programmatic dependent: it is scheduled when the kernel before it in the stream releases its
    // dependents (the attention kernels do so once their results are written) and waits for that kernel's completion
    // before it reads cache_len, so only the launch latency overlaps
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((threads + 127) / 128));
    cfg.blockDim = dim3(128);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, append_kernel, (char*)Kl, (char*)Vl, (const int32_t*)len_l, (const char*)Kq,
                                       (const char*)Vq, Hkv, T_q, capacity, row_bytes, threads, d_status);
    if (e != cudaSuccess) return e;
  }
  const int G = Hq / Hkv;
  const int rows = T_q * G;
  if (sizeof(T) == 2) {
    cudaError_t e = (plan.rows_per_cta == 128 && plan.share_sm)
                        ? launch_attn_tc3(s, Kl, Vl, capacity, len_l, Q, T_q, appended, scale, O, lse, part_o, part_ml,
                                          plan, d_status, stream)
                    : (plan.rows_per_cta == 128)
                        ? launch_attn_tc4(s, Kl, Vl, capacity, len_l, Q, T_q, Kq, Vq, scale, O, lse, part_o, part_ml,
                                          plan, d_status, stream)
                    : (plan.rows_per_cta == 256)
                        ? launch_attn_tc2(s, Kl, Vl, capacity, len_l, Q, T_q, appended, scale, O, lse, part_o, part_ml,
                                          plan, d_status, stream)
                        : launch_attn_mma(s, layer, Kl, Vl, capacity, len_l, Q, T_q, appended, scale, O, lse, part_o,
                                          part_ml, plan, stream);
    if (e != cudaSuccess) return e;
  } else {
    const int row_tiles = (rows + kSimtWarps - 1) / kSimtWarps;
    const long long blocks = (long long)Bt * Hkv * row_tiles * plan.n_splits;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    attn_simt_kernel<T, kHeadDim><<<(unsigned)blocks, kSimtWarps * 32, 0, stream>>>(
        Kl, Vl, len_l, (const T*)Q, (T*)O, lse, part_o, part_ml, Hq, Hkv, T_q, capacity, appended, scale,
        plan.n_splits, row_tiles);
  }
  if ((plan.n_splits > 1 || appended) && !(sizeof(T) == 2 && attn_merges_in_cluster(plan))) {
    const long long blocks = plan.n_splits > 1 ? (long long)((out_rows + 3) / 4) : 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(128);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    if (sizeof(T) == 2 && plan.rows_per_cta >= 128) {     // the tensor-memory kernels release their dependents early
      cfg.attrs = &attr;
      cfg.numAttrs = 1;
    }
    cudaError_t e = cudaLaunchKernelEx(&cfg, attn_finalize_kernel<T, kHeadDim>, (const float*)part_o,
                                       (const float2*)part_ml, (T*)O, lse, len_l, Bt, Hq, T_q, capacity, appended,
                                       plan.n_splits, (long long)out_rows);
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

cudaError_t launch_attn(const samkv_shape_t& s, int layer, void* Kc, void* Vc, int capacity, int32_t* cache_len,
                        const void* Q, int T_q, const void* Kq, const void* Vq, float scale, void* O, float* lse,
                        void* partial_ws, const AttnPlan& plan, int* d_status, cudaStream_t stream) {
  if (scale <= 0.f) scale = 1.0f / sqrtf((float)s.head_dim);
  if (s.dtype == SAMKV_BF16) {
    if (s.head_dim == 128)
      return launch_attn_t<__nv_bfloat16, 128>(s, layer, Kc, Vc, capacity, cache_len, Q, T_q, Kq, Vq, scale, O, lse,
                                               partial_ws, plan, d_status, stream);
    return launch_attn_t<__nv_bfloat16, 64>(s, layer, Kc, Vc, capacity, cache_len, Q, T_q, Kq, Vq, scale, O, lse,
                                            partial_ws, plan, d_status, stream);
  }
  if (s.head_dim == 128)
    return launch_attn_t<float, 128>(s, layer, Kc, Vc, capacity, cache_len, Q, T_q, Kq, Vq, scale, O, lse, partial_ws,
                                     plan, d_status, stream);
  return launch_attn_t<float, 64>(s, layer, Kc, Vc, capacity, cache_len, Q, T_q, Kq, Vq, scale, O, lse, partial_ws,
                                  plan, d_status, stream);
}

}  // namespace samkv
