// Block representatives (Sec. 3.2): Kbar[l, b, h, u, :] = mean of the key rows of unit u.  Query-independent, so
// it runs once when a document's cache is stored; scoring then reads d*e bytes per unit instead of per token.
#include "common.cuh"

namespace samkv {

constexpr int kMeanThreads = 256;

// One warp per unit.  A row is kLanes 16-byte vectors; a warp reads 32 / kLanes rows at once, each lane summing its
// vector position over every (32 / kLanes)-th row in fp32; the partial sums meet by shuffles.
template <typename T, int kHeadDim>
__global__ void __launch_bounds__(kMeanThreads)
block_means_kernel(const T* __restrict__ K, T* __restrict__ Kbar, const __grid_constant__ CtxTable ct, int L_tot,
                   int U_tot, long long n_units_all) {
  constexpr int kPerVec = ElemTraits<T>::kPerVec;
  constexpr int kLanes = kHeadDim / kPerVec;
  constexpr int kRowsAtOnce = 32 / kLanes;
  constexpr int kUnroll = 8;
  const int lane = threadIdx.x & 31;
  const int vec = lane % kLanes, rsub = lane / kLanes;
  const long long warp0 = ((long long)blockIdx.x * kMeanThreads + threadIdx.x) >> 5;
  const long long n_warps = ((long long)gridDim.x * kMeanThreads) >> 5;
  const int B = ct.block_size;
  for (long long w = warp0; w < n_units_all; w += n_warps) {
    const long long slab = w / U_tot;
    const int unit = (int)(w - slab * U_tot);
    const int c = find_segment(ct.unit_off, ct.n_ctx, unit);
    const int t0 = ct.ctx_off[c] + ((unit - ct.unit_off[c]) << ct.block_shift);
    const int n_tok = min(B, ct.ctx_off[c + 1] - t0);
    const char* src = reinterpret_cast<const char*>(K + ((size_t)slab * L_tot + t0) * kHeadDim) + vec * 16;
    float acc[kPerVec];
#pragma unroll
    for (int i = 0; i < kPerVec; ++i) acc[i] = 0.f;
    for (int r0 = rsub; r0 < n_tok; r0 += kRowsAtOnce * kUnroll) {
      uint4 v[kUnroll];
#pragma unroll
      for (int j = 0; j < kUnroll; ++j) {
        const int r = r0 + j * kRowsAtOnce;
        v[j] = r < n_tok ? ld_stream(src + (size_t)r * (kHeadDim * sizeof(T))) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int j = 0; j < kUnroll; ++j) {
        float f[kPerVec];
        ElemTraits<T>::unpack(v[j], f);
#pragma unroll
        for (int i = 0; i < kPerVec; ++i) acc[i] += f[i];
      }
    }
#pragma unroll
    for (int o = kLanes; o < 32; o <<= 1) {
#pragma unroll
      for (int i = 0; i < kPerVec; ++i) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);
    }
    if (rsub == 0) {
      const float inv = 1.0f / (float)n_tok;
#pragma unroll
      for (int i = 0; i < kPerVec; ++i) acc[i] *= inv;
      *reinterpret_cast<uint4*>(reinterpret_cast<char*>(Kbar + ((size_t)slab * U_tot + unit) * kHeadDim) + vec * 16) =
          ElemTraits<T>::pack(acc);
    }
  }
}

cudaError_t launch_block_means(const samkv_shape_t& s, const CtxTable& ct, const void* K, void* Kbar, int sm_count,
                               cudaStream_t stream) {
  const int L_tot = ct.ctx_off[ct.n_ctx], U_tot = ct.unit_off[ct.n_ctx];
  const long long n_units_all = (long long)s.n_layers * s.batch * s.n_kv_heads * U_tot;
  if (n_units_all == 0) return cudaSuccess;
  const long long want = (n_units_all + (kMeanThreads / 32) - 1) / (kMeanThreads / 32);
  const long long cap = (long long)sm_count * 8 * 4;                    // a few waves of 8 resident CTAs per SM
  const unsigned grid = (unsigned)(want < cap ? want : cap);
#define SAMKV_LAUNCH_MEANS(T, D)                                                                                     \
  block_means_kernel<T, D><<<grid, kMeanThreads, 0, stream>>>((const T*)K, (T*)Kbar, ct, L_tot, U_tot, n_units_all)
  if (s.dtype == SAMKV_BF16) {
    if (s.head_dim == 128) SAMKV_LAUNCH_MEANS(__nv_bfloat16, 128);
    else SAMKV_LAUNCH_MEANS(__nv_bfloat16, 64);
  } else {
    if (s.head_dim == 128) SAMKV_LAUNCH_MEANS(float, 128);
    else SAMKV_LAUNCH_MEANS(float, 64);
  }
#undef SAMKV_LAUNCH_MEANS
  return cudaGetLastError();
}

}  // namespace samkv
