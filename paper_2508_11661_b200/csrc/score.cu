// Scoring pass of SamKV: pooled query and personalised query (Eq. 1), then one streaming pass over
// every cached key row: s = <q_i, K_t>, block score = mean over the block's tokens (Sec. 3.2).
#include "common.cuh"

namespace samkv {

// ------------------------------------------------------------------------------------------------
// Block-wide sum of two values at once; blockDim.x is a multiple of 32 and at most 1024.
// Fixed reduction tree => bitwise reproducible.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float2 block_sum2(float a, float b, float2* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    a += __shfl_xor_sync(0xffffffffu, a, o);
    b += __shfl_xor_sync(0xffffffffu, b, o);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  __syncthreads();  // protect `red` from the previous use
  if (lane == 0) red[warp] = make_float2(a, b);
  __syncthreads();
  float2 r = make_float2(0.f, 0.f);
  for (int i = 0; i < nw; ++i) { r.x += red[i].x; r.y += red[i].y; }
  return r;
}

template <typename T>
__device__ __forceinline__ float load_as_float(const T* p);
template <>
__device__ __forceinline__ float load_as_float<float>(const float* p) { return *p; }
template <>
__device__ __forceinline__ float load_as_float<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// ------------------------------------------------------------------------------------------------
// Q_que = mean_t Q (Sec. 3.1), q_loc_j = mean_t Qloc_j, Eq. 1, then the mean over the G query heads
// of a KV group.  One CTA per (layer, batch, kv head); thread e owns element e of the head dimension.
// The sum over j != i is formed as (sum over all j) - (own term); fp32 throughout.
//   qhat [L*Bt, D, Hkv, d]
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void qhat_kernel(const T* __restrict__ Q, const T* __restrict__ Qloc, float* __restrict__ qhat, int T_q,
                            int T_loc, int Hq, int Hkv, int d, int D, int use_bias) {
  extern __shared__ float smem[];
  float* w = smem;                                        // [D] |cos| weights of the current query head
  float2* red = reinterpret_cast<float2*>(smem + D + (D & 1));  // [32]
  const int h = blockIdx.x % Hkv;
  const size_t lb = blockIdx.x / Hkv;
  const int e = threadIdx.x;
  const int G = Hq / Hkv;
  const bool bias = use_bias && Qloc != nullptr && D > 1;
  float* out = qhat + (lb * D * Hkv + h) * d + e;          // + i * Hkv * d
  const float inv_dm1 = bias ? 1.0f / (float)(D - 1) : 0.f;

  for (int g = 0; g < G; ++g) {
    const int hq = h * G + g;
    float qq = 0.f;
    for (int t = 0; t < T_q; ++t) qq += load_as_float(Q + ((lb * T_q + t) * Hq + hq) * d + e);
    qq = qq / (float)T_q;
    float S = 0.f;
    if (bias) {
      const float na2 = block_sum2(qq * qq, 0.f, red).x;
      for (int j = 0; j < D; ++j) {
        float ql = 0.f;
        for (int t = 0; t < T_loc; ++t) ql += load_as_float(Qloc + (((lb * D + j) * T_loc + t) * Hq + hq) * d + e);
        ql = ql / (float)T_loc;
        const float2 r = block_sum2(qq * ql, ql * ql, red);
        const float wj = (na2 > 0.f && r.y > 0.f) ? fabsf(r.x) / (sqrtf(na2) * sqrtf(r.y)) : 0.f;
        if (e == 0) w[j] = wj;
        S += wj * ql;
      }
      __syncthreads();
    }
    for (int i = 0; i < D; ++i) {
      float val = qq;
      if (bias) {
        float ql = 0.f;
        for (int t = 0; t < T_loc; ++t) ql += load_as_float(Qloc + (((lb * D + i) * T_loc + t) * Hq + hq) * d + e);
        ql = ql / (float)T_loc;
        val += (S - w[i] * ql) * inv_dm1;
      }
      float* o = out + (size_t)i * Hkv * d;
      const float acc = (g == 0) ? val : (*o + val);
      *o = (g == G - 1) ? acc / (float)G : acc;
    }
    __syncthreads();  // w[] is rewritten for the next query head
  }
}

cudaError_t launch_qhat(const samkv_shape_t& s, const void* Q, int T_q, const void* Qloc, int T_loc, int use_bias,
                        float* qhat, cudaStream_t stream) {
  const int blocks = s.n_layers * s.batch * s.n_kv_heads;
  const size_t smem = (size_t)(s.n_ctx + (s.n_ctx & 1)) * sizeof(float) + 32 * sizeof(float2);
  if (s.dtype == SAMKV_BF16)
    qhat_kernel<__nv_bfloat16><<<blocks, s.head_dim, smem, stream>>>(
        (const __nv_bfloat16*)Q, (const __nv_bfloat16*)Qloc, qhat, T_q, T_loc, s.n_q_heads, s.n_kv_heads, s.head_dim,
        s.n_ctx, use_bias);
  else
    qhat_kernel<float><<<blocks, s.head_dim, smem, stream>>>((const float*)Q, (const float*)Qloc, qhat, T_q, T_loc,
                                                             s.n_q_heads, s.n_kv_heads, s.head_dim, s.n_ctx, use_bias);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Streaming scorer.  A CTA owns a tile of kTile consecutive key rows of one context of one
// (layer, batch, kv head) slab.  A row is kLanes 16-byte vectors; kLanes adjacent threads read one
// row (fully coalesced), multiply with their slice of q_i held in registers and reduce with
// shuffles.  All of a thread's loads are issued before the first use, so a CTA keeps
// kTile * row_bytes (32 KB for bf16, d = 128) in flight.
// ------------------------------------------------------------------------------------------------
constexpr int kScoreThreads = 256;
constexpr int kScoreTile = 128;

struct TileTable {
  int tile_off[SAMKV_MAX_CTX + 1];  // prefix sum of ceil(L_c / kScoreTile)
};

template <typename T, int kHeadDim>
__global__ void __launch_bounds__(kScoreThreads)
score_kernel(const T* __restrict__ K, const float* __restrict__ qhat, float* __restrict__ scores,
             const __grid_constant__ CtxTable ct, const __grid_constant__ TileTable tt, int Hkv, int L_tot, int U_tot) {
  constexpr int kPerVec = ElemTraits<T>::kPerVec;
  constexpr int kLanes = kHeadDim / kPerVec;             // threads per row
  constexpr int kRowsPerPass = kScoreThreads / kLanes;
  constexpr int kPasses = kScoreTile / kRowsPerPass;
  static_assert(kLanes <= 32 && kPasses >= 1, "row must fit in a warp");

  __shared__ float s_tok[kScoreTile];

  const int tiles_per_slab = tt.tile_off[ct.n_ctx];
  const int tile = blockIdx.x % tiles_per_slab;
  const size_t slab = blockIdx.x / tiles_per_slab;         // (l * Bt + b) * Hkv + h
  const int c = find_segment(tt.tile_off, ct.n_ctx, tile);
  const int row0 = (tile - tt.tile_off[c]) * kScoreTile;    // first row of the tile inside its context
  const int L_c = ct.ctx_off[c + 1] - ct.ctx_off[c];
  const int rows = min(kScoreTile, L_c - row0);

  const int lane = threadIdx.x % kLanes;
  const int rsub = threadIdx.x / kLanes;
  const int h = (int)(slab % Hkv);
  const size_t lb = slab / Hkv;

  // this thread's slice of q_i
  float q[kPerVec];
  {
    const float* qp = qhat + ((lb * ct.n_ctx + c) * Hkv + h) * kHeadDim + lane * kPerVec;
#pragma unroll
    for (int i = 0; i < kPerVec; i += 4) {
      const float4 v = *reinterpret_cast<const float4*>(qp + i);
      q[i] = v.x; q[i + 1] = v.y; q[i + 2] = v.z; q[i + 3] = v.w;
    }
  }

  const T* base = K + (slab * L_tot + ct.ctx_off[c] + row0) * kHeadDim + lane * kPerVec;
  uint4 v[kPasses];
#pragma unroll
  for (int p = 0; p < kPasses; ++p) {
    const int r = p * kRowsPerPass + rsub;
    v[p] = (r < rows) ? ld_stream(base + (size_t)r * kHeadDim) : make_uint4(0, 0, 0, 0);
  }
#pragma unroll
  for (int p = 0; p < kPasses; ++p) {
    float f[kPerVec];
    ElemTraits<T>::unpack(v[p], f);
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < kPerVec; ++i) acc = fmaf(f[i], q[i], acc);
#pragma unroll
    for (int o = kLanes / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) s_tok[p * kRowsPerPass + rsub] = acc;
  }
  __syncthreads();

  // unit (block) scores: mean of the token scores of each unit, summed in token order
  const int B = ct.block_size;
  const int units = (rows + B - 1) >> ct.block_shift;
  if ((int)threadIdx.x < units) {
    const int a = threadIdx.x << ct.block_shift;
    const int n = min(B, rows - a);
    float sum = s_tok[a];
    for (int i = 1; i < n; ++i) sum += s_tok[a + i];
    scores[slab * U_tot + ct.unit_off[c] + (row0 >> ct.block_shift) + threadIdx.x] = (n == 1) ? sum : sum / (float)n;
  }
}

template <typename T, int kHeadDim>
static cudaError_t launch_score_t(const samkv_shape_t& s, const CtxTable& ct, const void* K, const float* qhat,
                                  float* scores, cudaStream_t stream) {
  TileTable tt;
  tt.tile_off[0] = 0;
  for (int c = 0; c < ct.n_ctx; ++c)
    tt.tile_off[c + 1] = tt.tile_off[c] + (ct.ctx_off[c + 1] - ct.ctx_off[c] + kScoreTile - 1) / kScoreTile;
  const long long slabs = (long long)s.n_layers * s.batch * s.n_kv_heads;
  const long long blocks = slabs * tt.tile_off[ct.n_ctx];
  if (blocks == 0) return cudaSuccess;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  score_kernel<T, kHeadDim><<<(unsigned)blocks, kScoreThreads, 0, stream>>>(
      (const T*)K, qhat, scores, ct, tt, s.n_kv_heads, ct.ctx_off[ct.n_ctx], ct.unit_off[ct.n_ctx]);
  return cudaGetLastError();
}

cudaError_t launch_score(const samkv_shape_t& s, const CtxTable& ct, const void* K, const float* qhat, float* scores,
                         cudaStream_t stream) {
  if (s.dtype == SAMKV_BF16) {
    if (s.head_dim == 128) return launch_score_t<__nv_bfloat16, 128>(s, ct, K, qhat, scores, stream);
    return launch_score_t<__nv_bfloat16, 64>(s, ct, K, qhat, scores, stream);
  }
  if (s.head_dim == 128) return launch_score_t<float, 128>(s, ct, K, qhat, scores, stream);
  return launch_score_t<float, 64>(s, ct, K, qhat, scores, stream);
}

}  // namespace samkv
