// Scoring pass of SamKV: pooled query and personalised query (Eq. 1), then one streaming pass over
// every cached key row: s = <q_i, K_t>, block score = mean over the block's tokens (Sec. 3.2).
#include "common.cuh"

namespace samkv {

template <typename T>
__device__ __forceinline__ float load_as_float(const T* p);
template <>
__device__ __forceinline__ float load_as_float<float>(const float* p) { return *p; }
template <>
__device__ __forceinline__ float load_as_float<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ------------------------------------------------------------------------------------------------
// Q_que = mean_t Q (Sec. 3.1), q_loc_j = mean_t Qloc_j, Eq. 1, then the mean over the G query heads
// of a KV group.  One CTA per (layer, batch, kv head) with one warp per query head of the group; a lane
// owns kEpl = d/32 consecutive elements (one vector load per row), so the cosines need warp shuffles
// only.  The kernel is latency-bound (a few KB per CTA), so independent work is batched: the local
// queries of kQhatBatch contexts are loaded and reduced together, and the GQA fold runs on chunks of
// contexts between two block barriers.  The sum over j != i is formed as (sum over all j) - (own
// term); fp32 throughout, fixed summation order.
//   qhat [L*Bt, D, Hkv, d]
// ------------------------------------------------------------------------------------------------
template <typename T>
constexpr int kQhatBatchOf = sizeof(T) == 2 ? 6 : 4;   // contexts whose local queries are in flight together
constexpr int kQhatFoldBytes = 24 * 1024;   // shared memory for one chunk of per-head Q^_i vectors
constexpr int kQhatLocalBytes = 24 * 1024;  // a group's local-query rows are staged in shared memory up to this size,
constexpr int kQhatFoldBytesStaged = 8 * 1024;   // with a smaller chunk of Q^_i vectors beside them

// A lane's kEpl consecutive elements of a row as loaded (one 4-, 8- or 16-byte load), and their conversion.  Keeping
// the loaded form in registers until the sum lets many rows be in flight without a float per element.
template <typename T, int kEpl> struct RowSlice;
template <> struct RowSlice<float, 4> { using Raw = float4; };
template <> struct RowSlice<float, 2> { using Raw = float2; };
template <> struct RowSlice<__nv_bfloat16, 4> { using Raw = uint2; };
template <> struct RowSlice<__nv_bfloat16, 2> { using Raw = uint32_t; };
__device__ __forceinline__ void slice_to_float(const float4& v, float* o) { o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w; }
__device__ __forceinline__ void slice_to_float(const float2& v, float* o) { o[0] = v.x; o[1] = v.y; }
__device__ __forceinline__ void slice_to_float(const uint2& v, float* o) {
  o[0] = bf16_lo(v.x); o[1] = bf16_hi(v.x); o[2] = bf16_lo(v.y); o[3] = bf16_hi(v.y);
}
__device__ __forceinline__ void slice_to_float(const uint32_t& v, float* o) { o[0] = bf16_lo(v); o[1] = bf16_hi(v); }

template <typename T, int kEpl>
__device__ __forceinline__ void load_row_slice(const T* p, float* out) {      // kEpl consecutive elements, one load
  slice_to_float(*reinterpret_cast<const typename RowSlice<T, kEpl>::Raw*>(p), out);
}

// kMaxThreads bounds G * 32; the register cap that comes with it keeps at least 7 / 3 / 1 CTAs of 128 / 256 / 1024
// threads on an SM, so that a grid of about a thousand CTAs is resident in one wave.
template <typename T, int kEpl, int kMaxThreads>
__global__ void __launch_bounds__(kMaxThreads, kMaxThreads == 128 ? 7 : (kMaxThreads == 256 ? 3 : 1))
qhat_kernel(const T* __restrict__ Q, const T* __restrict__ Qloc, float* __restrict__ qhat, int T_q,
                            int T_loc, int Hq, int Hkv, int D, int use_bias, int fold_ctx, int stage_local) {
  constexpr int d = kEpl * 32;
  constexpr int kQhatBatch = kQhatBatchOf<T>;
  extern __shared__ float smem[];
  pdl_launch_dependents();                   // the scoring kernel behind this one may start fetching key rows
  const int G = Hq / Hkv;
  float* w_all = smem;                       // [G][D] |cos| weights
  float* fold = smem + ((G * D + 3) & ~3);   // [fold_ctx][G][d] per-head Q^_i of a chunk of contexts (16-byte aligned)
  T* loc = reinterpret_cast<T*>(fold + fold_ctx * G * d);   // (stage_local) [D][T_loc][G][d] this group's local-query rows
  const int h = blockIdx.x % Hkv;
  const size_t lb = blockIdx.x / Hkv;
  const int g = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int hq = h * G + g;
  const bool bias = use_bias && Qloc != nullptr && D > 1;
  float* w = w_all + g * D;
  const size_t row_stride = (size_t)Hq * d;
  const bool staged = stage_local && use_bias && Qloc != nullptr && D > 1;
  if (staged) {
    // When the group's local-query rows are few, all of them are fetched into shared memory at once and in the
    // background (16-byte asynchronous copies), while the rows of Q are being pooled: both passes over them below
    // then cost no trip to memory.  A (context, row) holds the G heads of the group as one contiguous run.
    const int per_row = G * d * (int)sizeof(T) / 16;                 // 16-byte pieces of a run
    const int pieces = D * T_loc * per_row;
    for (int i = threadIdx.x; i < pieces; i += blockDim.x) {
      const int r = i / per_row, c = i - r * per_row;                // r = j * T_loc + t
      const char* src = reinterpret_cast<const char*>(Qloc + ((lb * D * T_loc + r) * Hq + (size_t)h * G) * d) + c * 16;
      const uint32_t dst = (uint32_t)__cvta_generic_to_shared(reinterpret_cast<char*>(loc) + (size_t)i * 16);
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  const size_t loc_stride = staged ? (size_t)G * d : row_stride;     // from a local row to the next one

  // mean over T_n rows, summed in row order; the loads of kRowsInFlight rows (a 16- or 32-byte register pair each) are issued before their sums
  constexpr int kRowsInFlight = sizeof(T) == 2 ? 16 : 8;
  auto pooled = [&](const T* base, int T_n, float* out) {
#pragma unroll
    for (int i = 0; i < kEpl; ++i) out[i] = 0.f;
    for (int t0 = 0; t0 < T_n; t0 += kRowsInFlight) {
      typename RowSlice<T, kEpl>::Raw r[kRowsInFlight];
#pragma unroll
      for (int u = 0; u < kRowsInFlight; ++u)
        if (t0 + u < T_n) r[u] = *reinterpret_cast<const typename RowSlice<T, kEpl>::Raw*>(base + (t0 + u) * row_stride + lane * kEpl);
#pragma unroll
      for (int u = 0; u < kRowsInFlight; ++u)
        if (t0 + u < T_n) {
          float f[kEpl];
          slice_to_float(r[u], f);
#pragma unroll
          for (int i = 0; i < kEpl; ++i) out[i] += f[i];
        }
    }
    if (T_n > 1) {
#pragma unroll
      for (int i = 0; i < kEpl; ++i) out[i] = out[i] / (float)T_n;
    }
  };
  auto qloc_row = [&](int j) -> const T* {
    return staged ? loc + ((size_t)j * T_loc * G + g) * d : Qloc + ((lb * D + j) * T_loc * Hq + hq) * d;
  };
  // local queries of contexts j0 .. j0 + kQhatBatch - 1 (zero past the last context): the rows of the batch are
  // loaded together, so that a batch costs one memory round trip per local row rather than one per context
  auto pooled_batch = [&](int j0, int j_end, float (*ql)[kEpl]) {
#pragma unroll
    for (int u = 0; u < kQhatBatch; ++u) {
#pragma unroll
      for (int i = 0; i < kEpl; ++i) ql[u][i] = 0.f;
    }
    for (int t = 0; t < T_loc; ++t) {
      float r[kQhatBatch][kEpl];
#pragma unroll
      for (int u = 0; u < kQhatBatch; ++u) {
        if (j0 + u < j_end) {
          load_row_slice<T, kEpl>(qloc_row(j0 + u) + t * loc_stride + lane * kEpl, r[u]);
        } else {
#pragma unroll
          for (int i = 0; i < kEpl; ++i) r[u][i] = 0.f;
        }
      }
#pragma unroll
      for (int u = 0; u < kQhatBatch; ++u) {
#pragma unroll
        for (int i = 0; i < kEpl; ++i) ql[u][i] += r[u][i];
      }
    }
    if (T_loc > 1) {
#pragma unroll
      for (int u = 0; u < kQhatBatch; ++u) {
#pragma unroll
        for (int i = 0; i < kEpl; ++i) ql[u][i] = ql[u][i] / (float)T_loc;
      }
    }
  };

  float qq[kEpl], S[kEpl];
  pooled(Q + (lb * T_q * Hq + hq) * d, T_q, qq);
#pragma unroll
  for (int i = 0; i < kEpl; ++i) S[i] = 0.f;
  if (staged) {
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();                                                 // every thread's pieces have landed
  }
  if (bias) {
    float na2 = 0.f;
#pragma unroll
    for (int i = 0; i < kEpl; ++i) na2 = fmaf(qq[i], qq[i], na2);
    na2 = warp_sum(na2);
    const float rnorm_a = na2 > 0.f ? rsqrtf(na2) : 0.f;
    for (int j0 = 0; j0 < D; j0 += kQhatBatch) {
      float ql[kQhatBatch][kEpl], dot[kQhatBatch], nb2[kQhatBatch];
      pooled_batch(j0, D, ql);
#pragma unroll
      for (int u = 0; u < kQhatBatch; ++u) {
        dot[u] = nb2[u] = 0.f;
#pragma unroll
        for (int i = 0; i < kEpl; ++i) { dot[u] = fmaf(qq[i], ql[u][i], dot[u]); nb2[u] = fmaf(ql[u][i], ql[u][i], nb2[u]); }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {                       // 2 * kQhatBatch independent shuffle chains
#pragma unroll
        for (int u = 0; u < kQhatBatch; ++u) {
          dot[u] += __shfl_xor_sync(0xffffffffu, dot[u], o);
          nb2[u] += __shfl_xor_sync(0xffffffffu, nb2[u], o);
        }
      }
#pragma unroll
      for (int u = 0; u < kQhatBatch; ++u) {                    // S accumulates in context order
        if (j0 + u < D) {
          // |cos| = |dot| / (|a| |b|) with reciprocal square roots (2 ulp each): a few instructions per context
          const float wj = (na2 > 0.f && nb2[u] > 0.f) ? fabsf(dot[u]) * rnorm_a * rsqrtf(nb2[u]) : 0.f;
          if (lane == 0) w[j0 + u] = wj;
#pragma unroll
          for (int i = 0; i < kEpl; ++i) S[i] = fmaf(wj, ql[u][i], S[i]);
        }
      }
    }
    __syncwarp();
  }
  const float inv_dm1 = bias ? 1.0f / (float)(D - 1) : 0.f;
  float* out = qhat + (lb * D * Hkv + h) * d;            // + i * Hkv * d
  for (int c0 = 0; c0 < D; c0 += fold_ctx) {
    const int nc = min(fold_ctx, D - c0);
    for (int ci0 = 0; ci0 < nc; ci0 += kQhatBatch) {
      float ql[kQhatBatch][kEpl];
      if (bias) pooled_batch(c0 + ci0, c0 + nc, ql);       // second read of the rows: served by the caches
#pragma unroll
      for (int u = 0; u < kQhatBatch; ++u) {
        if (ci0 + u < nc) {
          const float wi = bias ? w[c0 + ci0 + u] : 0.f;
#pragma unroll
          for (int i = 0; i < kEpl; ++i) {
            const float val = bias ? qq[i] + (S[i] - wi * ql[u][i]) * inv_dm1 : qq[i];
            fold[((ci0 + u) * G + g) * d + lane * kEpl + i] = val;
          }
        }
      }
    }
    __syncthreads();
    // mean over the G query heads of the group, summed in head order
    for (int e = threadIdx.x; e < nc * d; e += blockDim.x) {
      const int ci = e / d, x = e - ci * d;
      float acc = fold[(ci * G) * d + x];
      for (int gg = 1; gg < G; ++gg) acc += fold[(ci * G + gg) * d + x];
      out[(size_t)(c0 + ci) * Hkv * d + x] = acc / (float)G;
    }
    __syncthreads();
  }
}

cudaError_t launch_qhat(const samkv_shape_t& s, const void* Q, int T_q, const void* Qloc, int T_loc, int use_bias,
                        float* qhat, cudaStream_t stream) {
  const int blocks = s.n_layers * s.batch * s.n_kv_heads;
  const int G = s.n_q_heads / s.n_kv_heads;
  if (G > 32) return cudaErrorInvalidConfiguration;        // one warp per query head of a group
  const size_t elem = s.dtype == SAMKV_BF16 ? 2 : 4;
  const size_t local_bytes = (size_t)s.n_ctx * (T_loc > 0 ? T_loc : 0) * G * s.head_dim * elem;
  const int stage_local = use_bias && Qloc != nullptr && s.n_ctx > 1 && local_bytes <= (size_t)kQhatLocalBytes &&
                          (G * s.head_dim * elem) % 16 == 0;
  int fold_ctx = (stage_local ? kQhatFoldBytesStaged : kQhatFoldBytes) / (G * s.head_dim * (int)sizeof(float));
  fold_ctx = fold_ctx < 1 ? 1 : (fold_ctx > s.n_ctx ? s.n_ctx : fold_ctx);
  const size_t smem = (size_t)(((G * s.n_ctx + 3) & ~3) + fold_ctx * G * s.head_dim) * sizeof(float) +
                      (stage_local ? local_bytes : 0);
#define SAMKV_QHAT_N(T, EPL, N)                                                                                  \
  qhat_kernel<T, EPL, N><<<blocks, G * 32, smem, stream>>>((const T*)Q, (const T*)Qloc, qhat, T_q, T_loc,          \
                                                           s.n_q_heads, s.n_kv_heads, s.n_ctx, use_bias, fold_ctx, stage_local)
#define SAMKV_QHAT(T, EPL)                                                                                        \
  do {                                                                                                            \
    if (G <= 4) SAMKV_QHAT_N(T, EPL, 128);                                                                        \
    else if (G <= 8) SAMKV_QHAT_N(T, EPL, 256);                                                                   \
    else SAMKV_QHAT_N(T, EPL, 1024);                                                                              \
  } while (0)
  if (s.dtype == SAMKV_BF16) {
    if (s.head_dim == 128) SAMKV_QHAT(__nv_bfloat16, 4); else SAMKV_QHAT(__nv_bfloat16, 2);
  } else {
    if (s.head_dim == 128) SAMKV_QHAT(float, 4); else SAMKV_QHAT(float, 2);
  }
#undef SAMKV_QHAT_N
#undef SAMKV_QHAT
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Streaming scorer: one pass over every key row, s = <q_i, K_t>, unit score = mean over the unit.
//
// Persistent CTAs (two per SM) walk the list of tiles; a tile is up to 32 KB of consecutive key rows
// of one context of one (layer, batch, kv head) slab, i.e. one contiguous run in HBM.  A producer
// thread keeps a ring of kStages tiles in flight with bulk asynchronous copies (cp.async.bulk) that
// complete on mbarriers, so the bytes in flight do not depend on how fast CTAs are launched or how
// many registers the consumers hold.  Eight consumer warps read the tile from shared memory with
// conflict-free 16-byte loads: kLanes adjacent threads own one row, multiply it with their slice
// of q_i (registers) and reduce with shuffles.  Reduction order is fixed, so results are bitwise
// reproducible.  Every mbarrier wait is bounded; a timeout is recorded as a device check.
//
// kMulti: tiles of a cache whose contexts are short (the block representatives of Sec. 3.2: a few dozen
// rows per context).  A tile is then kRows consecutive rows of the slab whatever contexts they belong to
// (the concatenated axis is contiguous), the q_i of up to kMaxTileCtx contexts travel with it, and every
// row picks its own.  Needs block_size 1 (a unit never straddles a tile) and is chosen by the launcher.
// ------------------------------------------------------------------------------------------------
constexpr int kConsumerWarps = 8;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kStreamThreads = kConsumers + 32;      // + one producer warp
constexpr int kStages = 3;
constexpr int kTileBytesMax = 32 * 1024;
constexpr uint32_t kScoreSpinLimit = 1u << 22;
constexpr int kMaxTileCtx = 8;                       // contexts a tile of the kMulti variant may touch

struct TileTable {
  int tile_off[SAMKV_MAX_CTX + 1];  // prefix sum of ceil(L_c / rows per tile)
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
#ifdef SAMKV_DEBUG_CHECKS
// Debug build only: a test can shorten the wait limit and make the producer withhold the copies of its first tile,
// so that the consumers' wait for that tile runs out.  Nothing faults or hangs: every wait stays bounded.
__device__ uint32_t g_debug_spin_limit = 0;     // 0 = the regular limit
__device__ int g_debug_withhold_first_tile = 0;
#define SAMKV_SCORE_SPIN_LIMIT (g_debug_spin_limit ? g_debug_spin_limit : kScoreSpinLimit)
#else
#define SAMKV_SCORE_SPIN_LIMIT kScoreSpinLimit
#endif
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  const uint32_t limit = SAMKV_SCORE_SPIN_LIMIT;
  for (uint32_t i = 0; i < limit; ++i) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
  }
  return false;
}

template <typename T, int kHeadDim, bool kMulti>
__global__ void __launch_bounds__(kStreamThreads, 2)
score_stream_kernel(const T* __restrict__ K, const float* __restrict__ qhat, float* __restrict__ scores,
                    const __grid_constant__ CtxTable ct, const __grid_constant__ TileTable tt, int Hkv, int L_tot,
                    int U_tot, long long total_tiles, int* __restrict__ d_status) {
  constexpr int kPerVec = ElemTraits<T>::kPerVec;
  constexpr int kRowBytes = kHeadDim * (int)sizeof(T);
  constexpr int kRows = kTileBytesMax / kRowBytes;          // rows per tile
  constexpr int kChunks = kRowBytes / 16;                   // 16-byte chunks per row
  constexpr int kLanes = kChunks / 2;                       // threads per row: chunks `lane` and `lane + kLanes`
  constexpr int kRowsPerPass = kConsumers / kLanes;
  constexpr int kPasses = kRows / kRowsPerPass;
  constexpr int kQBytes = kHeadDim * (int)sizeof(float);
  static_assert(kLanes >= 1 && kLanes <= 32 && kPasses >= 1 && kRows % 64 == 0, "tile shape");

  constexpr int kQPerStage = kMulti ? kMaxTileCtx : 1;      // q_i vectors that travel with a tile

  // shared memory: [tiles kStages x 32 KB][q kStages x kQPerStage x kQBytes][token scores kStages x kRows]
  //                [meta kStages x 3 int4][barriers]
  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* tiles = smem_raw;
  float* s_q = reinterpret_cast<float*>(smem_raw + kStages * kTileBytesMax);
  float* s_tok = s_q + kStages * kQPerStage * kHeadDim;
  // {rows, score offset lo, hi, contexts in the tile}, then (kMulti) the tile row at which each of the tile's
  // contexts ends, two int4
  int4* s_meta = reinterpret_cast<int4*>(s_tok + kStages * kRows);
  uint64_t* bars = reinterpret_cast<uint64_t*>(s_meta + 3 * kStages);       // full[kStages], empty[kStages]
  volatile int* s_fail = reinterpret_cast<volatile int*>(bars + 2 * kStages);
  const uint32_t full0 = smem_addr(bars), empty0 = smem_addr(bars + kStages);

  const int tid = threadIdx.x;
  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full0 + 8 * i), "r"(1) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty0 + 8 * i), "r"(kConsumerWarps) : "memory");
    }
    *s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  const long long first = blockIdx.x, stride = gridDim.x;

  if (tid >= kConsumers) {
    // ===== producer: one thread locates each tile and issues its bulk copies (key rows + q_i) =====
    if (tid == kConsumers) {
      const int tiles_per_slab = kMulti ? (L_tot + kRows - 1) / kRows : tt.tile_off[ct.n_ctx];
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      long long n = 0;
      bool ok = true;
      for (long long g = first; g < total_tiles; g += stride, ++n) {
        const int stage = (int)(n % kStages);
        const uint32_t round = (uint32_t)(n / kStages);
        if (!mbar_wait_bounded(empty0 + 8 * stage, (round & 1) ^ 1)) { ok = false; break; }
        const size_t slab = (size_t)(g / tiles_per_slab);           // (l * Bt + b) * Hkv + h
        const int tile = (int)(g % tiles_per_slab);
        int c, row0, rows, nq = 1;                                  // first context, first row (slab axis if kMulti)
        long long out;
        const T* src;
        if constexpr (kMulti) {
          row0 = tile * kRows;
          rows = min(kRows, L_tot - row0);
          c = find_segment(ct.ctx_off, ct.n_ctx, row0);
          nq = find_segment(ct.ctx_off, ct.n_ctx, row0 + rows - 1) - c + 1;       // <= kMaxTileCtx: the launcher checked
          int ends[kMaxTileCtx];
#pragma unroll
          for (int k = 0; k < kMaxTileCtx; ++k) ends[k] = k < nq - 1 ? ct.ctx_off[c + k + 1] - row0 : 0x7fffffff;
          s_meta[3 * stage + 1] = make_int4(ends[0], ends[1], ends[2], ends[3]);
          s_meta[3 * stage + 2] = make_int4(ends[4], ends[5], ends[6], ends[7]);
          out = (long long)slab * U_tot + row0;                     // block_size 1: a row is a unit
          src = K + (slab * L_tot + row0) * kHeadDim;
        } else {
          c = find_segment(tt.tile_off, ct.n_ctx, tile);
          row0 = (tile - tt.tile_off[c]) * kRows;                   // first row of the tile inside its context
          rows = min(kRows, ct.ctx_off[c + 1] - ct.ctx_off[c] - row0);
          out = (long long)slab * U_tot + ct.unit_off[c] + (row0 >> ct.block_shift);
          src = K + (slab * L_tot + ct.ctx_off[c] + row0) * kHeadDim;
        }
        s_meta[3 * stage] = make_int4(rows, (int)(out & 0xffffffffLL), (int)(out >> 32), nq);
        const uint32_t bytes = (uint32_t)rows * kRowBytes;
        const float* qsrc = qhat + (((slab / Hkv) * ct.n_ctx + c) * Hkv + slab % Hkv) * kHeadDim;
        const uint32_t bar = full0 + 8 * stage;
#ifdef SAMKV_DEBUG_CHECKS
        if (g_debug_withhold_first_tile && n == 0) continue;      // the consumers' wait for this tile runs out
#endif
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes + nq * kQBytes) : "memory");
        asm volatile(
            "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
            ::"r"(smem_addr(tiles + stage * kTileBytesMax)), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
        // The key rows were written before the pooled-query kernel started; its q_i are complete only after this
        // (the kernel is launched while that one is still running).
        if (n == 0) pdl_wait();
        for (int k = 0; k < nq; ++k)                                // q_i of context c + k (one copy unless kMulti)
          asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                       ::"r"(smem_addr(s_q + (stage * kQPerStage + k) * kHeadDim)), "l"(qsrc + (size_t)k * Hkv * kHeadDim),
                       "r"(kQBytes), "r"(bar) : "memory");
      }
      // do not leave while a copy of ours may still be landing: wait (bounded) for the last copy of every stage
      for (long long k = (n > kStages ? n - kStages : 0); k < n; ++k)
        if (!mbar_wait_bounded(full0 + 8 * (int)(k % kStages), (uint32_t)((k / kStages) & 1))) ok = false;
      if (!ok && d_status != nullptr) atomicMax(d_status, (int)CHECK_WAIT_TIMEOUT);
    }
    return;
  }

  // ===== consumers =====
  const int lane = tid % kLanes;
  const int rsub = tid / kLanes;

  long long n = 0;
  for (long long g = first; g < total_tiles; g += stride, ++n) {
    const int stage = (int)(n % kStages);
    const uint32_t round = (uint32_t)(n / kStages);
    // A timeout is only recorded here; every consumer still reaches the named barrier below and they all
    // leave together after it, so a failure can never strand a thread at a barrier.
    if (!mbar_wait_bounded(full0 + 8 * stage, round & 1)) {
      *s_fail = 1;
      if (d_status != nullptr) atomicMax(d_status, (int)CHECK_WAIT_TIMEOUT);
    }
    const int4 meta = s_meta[3 * stage];
    const int rows = meta.x;
    const unsigned char* tile = tiles + stage * kTileBytesMax + lane * 16;
    float* st = s_tok + stage * kRows;
    uint4 v0[kPasses], v1[kPasses];
#pragma unroll
    for (int p = 0; p < kPasses; ++p) {
      const int r = p * kRowsPerPass + rsub;
      if (r < rows) {
        v0[p] = *reinterpret_cast<const uint4*>(tile + (size_t)r * kRowBytes);
        v1[p] = *reinterpret_cast<const uint4*>(tile + (size_t)r * kRowBytes + kLanes * 16);
      } else {
        v0[p] = v1[p] = make_uint4(0, 0, 0, 0);
      }
    }
    // this thread's two slices of a q_i: elements of chunks `lane` and `lane + kLanes`
    float q[2 * kPerVec];
    auto load_q = [&](int k) {
      const float* qs = s_q + (stage * kQPerStage + k) * kHeadDim;
#pragma unroll
      for (int i = 0; i < kPerVec; i += 4) {
        const float4 a = *reinterpret_cast<const float4*>(qs + lane * kPerVec + i);
        const float4 b = *reinterpret_cast<const float4*>(qs + (lane + kLanes) * kPerVec + i);
        q[i] = a.x; q[i + 1] = a.y; q[i + 2] = a.z; q[i + 3] = a.w;
        q[kPerVec + i] = b.x; q[kPerVec + i + 1] = b.y; q[kPerVec + i + 2] = b.z; q[kPerVec + i + 3] = b.w;
      }
    };
    int ends[kMaxTileCtx];
    int k_have = 0;
    load_q(0);
    if constexpr (kMulti) {
      const int4 e0 = s_meta[3 * stage + 1], e1 = s_meta[3 * stage + 2];
      ends[0] = e0.x; ends[1] = e0.y; ends[2] = e0.z; ends[3] = e0.w;
      ends[4] = e1.x; ends[5] = e1.y; ends[6] = e1.z; ends[7] = e1.w;
    } else {
      // the tile, q_i and meta are in registers: hand the stage back to the producer
      __syncwarp();
      if ((tid & 31) == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty0 + 8 * stage) : "memory");
    }
#pragma unroll
    for (int p = 0; p < kPasses; ++p) {
      if constexpr (kMulti) {                                     // the q_i of this row's context
        const int r = p * kRowsPerPass + rsub;
        int k = 0;
#pragma unroll
        for (int j = 0; j < kMaxTileCtx - 1; ++j) k += (ends[j] <= r) ? 1 : 0;
        if (k != k_have) { load_q(k); k_have = k; }               // same k for the kLanes threads of a row
      }
      float f[kPerVec], g2[kPerVec];
      ElemTraits<T>::unpack(v0[p], f);
      ElemTraits<T>::unpack(v1[p], g2);
      float acc = 0.f;
#pragma unroll
      for (int i = 0; i < kPerVec; ++i) acc = fmaf(f[i], q[i], acc);
#pragma unroll
      for (int i = 0; i < kPerVec; ++i) acc = fmaf(g2[i], q[kPerVec + i], acc);
#pragma unroll
      for (int o = kLanes / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      if (lane == 0) st[p * kRowsPerPass + rsub] = acc;
    }
    if constexpr (kMulti) {                                       // the q_i were read above: now the stage is free
      __syncwarp();
      if ((tid & 31) == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty0 + 8 * stage) : "memory");
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
    if (*s_fail) break;      // written only by consumers, before they arrived at the barrier: uniform

    // unit (block) scores: mean of the token scores of each unit, summed in token order
    const int Bsz = ct.block_size;
    const int units = (rows + Bsz - 1) >> ct.block_shift;
    if (tid < units) {
      const int a = tid << ct.block_shift;
      const int cnt = min(Bsz, rows - a);
      float sum = st[a];
      for (int i = 1; i < cnt; ++i) sum += st[a + i];
      const long long out = ((long long)meta.z << 32) | (unsigned int)meta.y;
      scores[out + tid] = (cnt == 1) ? sum : sum / (float)cnt;
    }
  }
}

template <typename T, int kHeadDim, bool kMulti>
static cudaError_t launch_score_variant(const samkv_shape_t& s, const CtxTable& ct, const TileTable& tt,
                                        long long tiles_per_slab, const void* K, const float* qhat, float* scores,
                                        int* d_status, cudaStream_t stream) {
  constexpr int kRows = kTileBytesMax / (kHeadDim * (int)sizeof(T));
  constexpr int kQPerStage = kMulti ? kMaxTileCtx : 1;
  const long long slabs = (long long)s.n_layers * s.batch * s.n_kv_heads;
  const long long total_tiles = slabs * tiles_per_slab;
  if (total_tiles == 0) return cudaSuccess;
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  const size_t smem = (size_t)kStages * (kTileBytesMax + kQPerStage * kHeadDim * sizeof(float) + kRows * sizeof(float) + 48) +
                      2 * kStages * 8 + 16;
  auto kern = score_stream_kernel<T, kHeadDim, kMulti>;
  e = ensure_dynamic_smem<100 + kHeadDim + (kMulti ? 1 : 0)>(kern, (int)smem);
  if (e != cudaSuccess) return e;
  const long long grid = total_tiles < 2LL * sms ? total_tiles : 2LL * sms;
  // Launched so that it may begin while the kernel before it in the stream (always the pooled-query kernel of the
  // same call) is finishing: the producer fetches its first key rows, then waits for that kernel's results.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kStreamThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, (const T*)K, qhat, scores, ct, tt, (int)s.n_kv_heads, (int)ct.ctx_off[ct.n_ctx],
                            (int)ct.unit_off[ct.n_ctx], total_tiles, d_status);
}

template <typename T, int kHeadDim>
static cudaError_t launch_score_t(const samkv_shape_t& s, const CtxTable& ct, const void* K, const float* qhat,
                                  float* scores, int* d_status, cudaStream_t stream) {
  constexpr int kRows = kTileBytesMax / (kHeadDim * (int)sizeof(T));
  TileTable tt;
  tt.tile_off[0] = 0;
  for (int c = 0; c < ct.n_ctx; ++c)
    tt.tile_off[c + 1] = tt.tile_off[c] + (ct.ctx_off[c + 1] - ct.ctx_off[c] + kRows - 1) / kRows;
  // Short contexts (block representatives): tiles that ignore context boundaries, when fewer of them cover the slab
  // and none touches more than kMaxTileCtx contexts.
  const int L_tot = ct.ctx_off[ct.n_ctx];
  const int flat_tiles = (L_tot + kRows - 1) / kRows;
  bool multi = ct.block_shift == 0 && ct.n_ctx > 1 && flat_tiles < tt.tile_off[ct.n_ctx] &&
               (long long)L_tot < 2LL * kRows * ct.n_ctx;
  for (int t = 0, c = 0; multi && t < flat_tiles; ++t) {
    const int first = t * kRows, last = (first + kRows < L_tot ? first + kRows : L_tot) - 1;
    while (ct.ctx_off[c + 1] <= first) ++c;                  // context of the tile's first row (skips empty contexts)
    int c_last = c;
    while (ct.ctx_off[c_last + 1] <= last) ++c_last;
    if (c_last - c + 1 > kMaxTileCtx) multi = false;
  }
  if (multi) return launch_score_variant<T, kHeadDim, true>(s, ct, tt, flat_tiles, K, qhat, scores, d_status, stream);
  return launch_score_variant<T, kHeadDim, false>(s, ct, tt, tt.tile_off[ct.n_ctx], K, qhat, scores, d_status, stream);
}

cudaError_t launch_score(const samkv_shape_t& s, const CtxTable& ct, const void* K, const float* qhat, float* scores,
                         int* d_status, cudaStream_t stream) {
  if (s.dtype == SAMKV_BF16) {
    if (s.head_dim == 128) return launch_score_t<__nv_bfloat16, 128>(s, ct, K, qhat, scores, d_status, stream);
    return launch_score_t<__nv_bfloat16, 64>(s, ct, K, qhat, scores, d_status, stream);
  }
  if (s.head_dim == 128) return launch_score_t<float, 128>(s, ct, K, qhat, scores, d_status, stream);
  return launch_score_t<float, 64>(s, ct, K, qhat, scores, d_status, stream);
}

#ifdef SAMKV_DEBUG_CHECKS
cudaError_t debug_set_score_wait(uint32_t spin_limit, int withhold_first_tile, cudaStream_t stream) {
  cudaError_t e = cudaMemcpyToSymbolAsync(g_debug_spin_limit, &spin_limit, sizeof(spin_limit), 0, cudaMemcpyHostToDevice, stream);
  if (e != cudaSuccess) return e;
  return cudaMemcpyToSymbolAsync(g_debug_withhold_first_tile, &withhold_first_tile, sizeof(int), 0, cudaMemcpyHostToDevice,
                                 stream);
}
#endif

}  // namespace samkv
