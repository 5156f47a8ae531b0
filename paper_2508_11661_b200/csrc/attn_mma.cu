// bf16 tensor-core attention over the compact cache (Sec. 3.3), split-KV with online softmax.
//
// A CTA owns kWarps*16 packed query rows of one (batch, kv head) and one KV split; every warp owns 16
// rows.  K/V tiles of 64 slots are staged in shared memory with cp.async (two stages, 16-byte chunks
// XOR-swizzled so ldmatrix is bank-conflict free).  QK^T and PV run on mma.sync m16n8k16 with fp32
// accumulators; the softmax is computed in fp32 in the exp2 domain; probabilities are rounded to
// bf16 for the PV product.
#include <math.h>

#include "common.cuh"

namespace samkv {

constexpr int kBN = 64;            // KV slots per tile
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;   // src-size 0 => the 16 bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// byte offset of 16-byte chunk `chunk` of row `row` in a swizzled tile with kChunks chunks per row
template <int kChunks>
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  return (uint32_t)((row * kChunks + (chunk ^ (row & 7))) * 16);
}

template <int kHeadDim, int kWarps>
__global__ void __launch_bounds__(kWarps * 32)
attn_mma_kernel(const __nv_bfloat16* __restrict__ Kc, const __nv_bfloat16* __restrict__ Vc,
                const int32_t* __restrict__ cache_len, const __nv_bfloat16* __restrict__ Q,
                __nv_bfloat16* __restrict__ O, float* __restrict__ lse, float* __restrict__ part_o,
                float2* __restrict__ part_ml, int Hq, int Hkv, int T_q, int capacity, int appended, float scale,
                int n_splits, int row_tiles) {
  constexpr int kBM = kWarps * 16;
  constexpr int kChunks = kHeadDim / 8;          // 16-byte chunks per row
  constexpr int kThreads = kWarps * 32;
  constexpr int kTileBytes = kBN * kHeadDim * 2;
  constexpr int kDTiles = kHeadDim / 8;           // n-tiles of the output
  constexpr int kKSteps = kHeadDim / 16;          // k-steps of QK^T

  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* sQ = smem_raw;                               // kBM rows
  unsigned char* sK = sQ + kBM * kHeadDim * 2;                 // 2 stages
  unsigned char* sV = sK + 2 * kTileBytes;                     // 2 stages

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int grp = lane >> 2, qd = lane & 3;
  const int G = Hq / Hkv;
  const int split = blockIdx.x % n_splits;
  const int rtile = (blockIdx.x / n_splits) % row_tiles;
  const int bh = blockIdx.x / (n_splits * row_tiles);
  const int h = bh % Hkv, b = bh / Hkv;
  const int rows_total = T_q * G;
  const int row_base = rtile * kBM;

  int len = cache_len[b];
  len = max(0, min(len, capacity));
  const int n_app = (appended && len + T_q <= capacity) ? T_q : 0;
  const int total = len + n_app;
  const int last_row = min(row_base + kBM, rows_total) - 1;
  const int cta_visible = len + (n_app ? last_row / G + 1 : 0);          // widest row of this CTA
  const int n_tiles = (total + kBN - 1) / kBN;
  const int tps = (n_tiles + n_splits - 1) / n_splits;
  const int tile0 = split * tps;
  const int tile1 = min(min(tile0 + tps, n_tiles), (cta_visible + kBN - 1) / kBN);

  // ---- stage Q (zero rows beyond rows_total) ----
  for (int i = tid; i < kBM * kChunks; i += kThreads) {
    const int r = i / kChunks, c = i % kChunks;
    const int rr = row_base + r;
    const bool ok = rr < rows_total;
    const int t = ok ? rr / G : 0, g = ok ? rr % G : 0;
    const __nv_bfloat16* src = Q + (((size_t)b * T_q + t) * Hq + h * G + g) * kHeadDim + c * 8;
    cp_async16(smem_u32(sQ) + swz<kChunks>(r, c), src, ok);
  }
  const __nv_bfloat16* kbase = Kc + (size_t)bh * capacity * kHeadDim;
  const __nv_bfloat16* vbase = Vc + (size_t)bh * capacity * kHeadDim;
  auto load_tile = [&](int tile, int stage) {
    const int j0 = tile * kBN;
    for (int i = tid; i < kBN * kChunks; i += kThreads) {
      const int r = i / kChunks, c = i % kChunks;
      const bool ok = j0 + r < total;
      const size_t off = (size_t)(ok ? j0 + r : 0) * kHeadDim + c * 8;
      const uint32_t d = stage * kTileBytes + swz<kChunks>(r, c);
      cp_async16(smem_u32(sK) + d, kbase + off, ok);
      cp_async16(smem_u32(sV) + d, vbase + off, ok);
    }
  };
  if (tile0 < tile1) load_tile(tile0, 0);
  cp_async_commit();

  // ---- per-thread state ----
  const int r0 = row_base + warp * 16 + grp;       // rows r0 and r0 + 8
  const int vis0 = len + (n_app ? min(r0, rows_total - 1) / G + 1 : 0);
  const int vis1 = len + (n_app ? min(r0 + 8, rows_total - 1) / G + 1 : 0);
  const float sl2 = scale * kLog2e;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  float o[kDTiles][4];
#pragma unroll
  for (int i = 0; i < kDTiles; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  uint32_t qf[kKSteps][4];

  for (int tile = tile0; tile < tile1; ++tile) {
    const int stage = (tile - tile0) & 1;
    if (tile + 1 < tile1) load_tile(tile + 1, stage ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if (tile == tile0) {
#pragma unroll
      for (int ks = 0; ks < kKSteps; ++ks) {
        const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int chunk = ks * 2 + (lane >> 4);
        ldsm_x4(smem_u32(sQ) + swz<kChunks>(row, chunk), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
      }
    }
    const uint32_t sKs = smem_u32(sK) + stage * kTileBytes;
    const uint32_t sVs = smem_u32(sV) + stage * kTileBytes;

    // ---- S = Q K^T ----
    float s[kBN / 8][4];
#pragma unroll
    for (int i = 0; i < kBN / 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < kKSteps; ++ks) {
#pragma unroll
      for (int np = 0; np < kBN / 16; ++np) {
        const int mi = lane >> 3;
        const int row = np * 16 + (lane & 7) + (mi >> 1) * 8;
        const int chunk = ks * 2 + (mi & 1);
        uint32_t b0, b1, b2, b3;
        ldsm_x4(sKs + swz<kChunks>(row, chunk), b0, b1, b2, b3);
        mma_bf16(s[np * 2], qf[ks], b0, b1);
        mma_bf16(s[np * 2 + 1], qf[ks], b2, b3);
      }
    }

    // ---- mask (only tiles that reach past the shortest visible range of this warp's rows) ----
    const int j0 = tile * kBN;
    if (j0 + kBN > min(vis0, vis1)) {
#pragma unroll
      for (int nt = 0; nt < kBN / 8; ++nt) {
        const int j = j0 + nt * 8 + qd * 2;
        if (j >= vis0) s[nt][0] = -INFINITY;
        if (j + 1 >= vis0) s[nt][1] = -INFINITY;
        if (j >= vis1) s[nt][2] = -INFINITY;
        if (j + 1 >= vis1) s[nt][3] = -INFINITY;
      }
    }

    // ---- online softmax (exp2 domain) ----
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < kBN / 8; ++nt) {
      mx0 = fmaxf(mx0, fmaxf(s[nt][0], s[nt][1]));
      mx1 = fmaxf(mx1, fmaxf(s[nt][2], s[nt][3]));
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float mn0 = fmaxf(m0, mx0 * sl2), mn1 = fmaxf(m1, mx1 * sl2);
    const float mu0 = (mn0 == -INFINITY) ? 0.f : mn0, mu1 = (mn1 == -INFINITY) ? 0.f : mn1;
    const float c0 = fast_exp2(m0 - mu0), c1 = fast_exp2(m1 - mu1);
    m0 = mn0; m1 = mn1;
    float ps0 = 0.f, ps1 = 0.f;
    uint32_t pf[kBN / 16][4];
#pragma unroll
    for (int nt = 0; nt < kBN / 8; ++nt) {
      const float p0 = fast_exp2(fmaf(s[nt][0], sl2, -mu0));
      const float p1 = fast_exp2(fmaf(s[nt][1], sl2, -mu0));
      const float p2 = fast_exp2(fmaf(s[nt][2], sl2, -mu1));
      const float p3 = fast_exp2(fmaf(s[nt][3], sl2, -mu1));
      ps0 += p0 + p1;
      ps1 += p2 + p3;
      pf[nt >> 1][(nt & 1) * 2] = pack_bf16(p0, p1);
      pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
    l0 = l0 * c0 + ps0;
    l1 = l1 * c1 + ps1;
#pragma unroll
    for (int dt = 0; dt < kDTiles; ++dt) {
      o[dt][0] *= c0; o[dt][1] *= c0; o[dt][2] *= c1; o[dt][3] *= c1;
    }

    // ---- O += P V ----
#pragma unroll
    for (int ks = 0; ks < kBN / 16; ++ks) {
#pragma unroll
      for (int dp = 0; dp < kDTiles / 2; ++dp) {
        const int mi = lane >> 3;
        const int row = ks * 16 + (lane & 7) + (mi & 1) * 8;
        const int chunk = dp * 2 + (mi >> 1);
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(sVs + swz<kChunks>(row, chunk), b0, b1, b2, b3);
        mma_bf16(o[dp * 2], pf[ks], b0, b1);
        mma_bf16(o[dp * 2 + 1], pf[ks], b2, b3);
      }
    }
    __syncthreads();   // the stage is refilled by the next iteration's prefetch
  }
  cp_async_wait<0>();

  // ---- finish: reduce row sums across the quad, write ----
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int rr = r0 + half * 8;
    if (rr >= rows_total) continue;
    const int t = rr / G, hq = h * G + rr % G;
    const size_t orow = ((size_t)b * T_q + t) * Hq + hq;
    const float l = half ? l1 : l0;
    const float m = half ? m1 : m0;
    if (n_splits == 1) {
      const float inv = l > 0.f ? 1.0f / l : 0.f;
      __nv_bfloat16* op = O + orow * kHeadDim + qd * 2;
#pragma unroll
      for (int dt = 0; dt < kDTiles; ++dt)
        *reinterpret_cast<uint32_t*>(op + dt * 8) = pack_bf16(o[dt][half * 2] * inv, o[dt][half * 2 + 1] * inv);
      if (lse != nullptr && qd == 0) lse[((size_t)b * Hq + hq) * T_q + t] = l > 0.f ? m * kLn2 + logf(l) : -INFINITY;
    } else {
      float* po = part_o + (orow * n_splits + split) * kHeadDim + qd * 2;
#pragma unroll
      for (int dt = 0; dt < kDTiles; ++dt)
        *reinterpret_cast<float2*>(po + dt * 8) = make_float2(o[dt][half * 2], o[dt][half * 2 + 1]);
      if (qd == 0) part_ml[orow * n_splits + split] = make_float2(m * kLn2, l);
    }
  }
}

template <int kHeadDim, int kWarps>
static cudaError_t launch_mma_t(const samkv_shape_t& s, const void* Kc, const void* Vc, int capacity,
                                const int32_t* cache_len, const void* Q, int T_q, int appended, float scale, void* O,
                                float* lse, float* part_o, float2* part_ml, const AttnPlan& plan, cudaStream_t stream) {
  constexpr int kBM = kWarps * 16;
  const int G = s.n_q_heads / s.n_kv_heads;
  const int rows = T_q * G;
  const int row_tiles = (rows + kBM - 1) / kBM;
  const long long blocks = (long long)s.batch * s.n_kv_heads * row_tiles * plan.n_splits;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  const int smem = kBM * kHeadDim * 2 + 4 * kBN * kHeadDim * 2;
  auto kern = attn_mma_kernel<kHeadDim, kWarps>;
  if (smem > 48 * 1024) {
    cudaError_t e = ensure_dynamic_smem<2000 + kHeadDim * 16 + kWarps>(kern, smem);
    if (e != cudaSuccess) return e;
  }
  kern<<<(unsigned)blocks, kWarps * 32, smem, stream>>>(
      (const __nv_bfloat16*)Kc, (const __nv_bfloat16*)Vc, cache_len, (const __nv_bfloat16*)Q, (__nv_bfloat16*)O, lse,
      part_o, part_ml, s.n_q_heads, s.n_kv_heads, T_q, capacity, appended, scale, plan.n_splits, row_tiles);
  return cudaGetLastError();
}

cudaError_t launch_attn_mma(const samkv_shape_t& s, int layer, const void* Kc, const void* Vc, int capacity,
                            const int32_t* cache_len, const void* Q, int T_q, int appended, float scale, void* O,
                            float* lse, float* part_o, float2* part_ml, const AttnPlan& plan, cudaStream_t stream) {
  (void)layer;
#define SAMKV_MMA(HD, W) \
  return launch_mma_t<HD, W>(s, Kc, Vc, capacity, cache_len, Q, T_q, appended, scale, O, lse, part_o, part_ml, plan, stream)
  if (s.head_dim == 128) {
    if (plan.rows_per_cta == 128) SAMKV_MMA(128, 8);
    if (plan.rows_per_cta == 64) SAMKV_MMA(128, 4);
    SAMKV_MMA(128, 1);
  } else {
    if (plan.rows_per_cta == 128) SAMKV_MMA(64, 8);
    if (plan.rows_per_cta == 64) SAMKV_MMA(64, 4);
    SAMKV_MMA(64, 1);
  }
#undef SAMKV_MMA
}

}  // namespace samkv
