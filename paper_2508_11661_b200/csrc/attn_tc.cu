// bf16 attention over the compact cache on the 5th-generation tensor cores (tcgen05), for query
// chunks with at least 128 packed rows per KV head (Sec. 3.3: the re-prefill of the user query).
//
// A CTA of 128 threads owns 128 packed query rows (row r = token r / G, group member r % G) of one
// (batch, kv head) and one KV split.  Per 64-slot KV tile:
//   S = Q K^T      tcgen05.mma, M=128 N=64 K=16 x 8, operands in shared memory (K-major, 128-byte
//                  swizzle), accumulator in tensor memory (64 columns)
//   softmax        thread t owns row t: it reads its S row from tensor memory (tcgen05.ld), so row
//                  max / sum need no shuffles; P is rounded to bf16 and written to shared memory
//   O += P V       tcgen05.mma, M=128 N=128 K=16 x 4, V read as the MN-major B operand straight from
//                  its natural [slot][d] layout; O lives in tensor memory (128 columns) and is
//                  rescaled there only when a row maximum grows by more than 2^8
// MMAs are issued by one thread and complete on an mbarrier (tcgen05.commit).  K/V tiles are
// staged by cp.async (rows past the visible range are zero-filled) in two-stage rings; two CTAs share
// an SM so one CTA's softmax overlaps the other's MMAs.  Every wait is bounded: on a timeout the
// kernel records a device check, frees its tensor memory and returns.
#include <math.h>

#include "common.cuh"

namespace samkv {

namespace tc {

constexpr int kBM = 128;       // packed query rows per CTA
constexpr int kBN = 64;        // KV slots per tile
constexpr int kD = 128;        // head dimension
constexpr int kThreads = 128;
constexpr int kQBytes = kBM * kD * 2;          // 32 KB: two 64-element blocks of [128 rows][128 B]
constexpr int kTileBytes = kBN * kD * 2;       // 16 KB: two 64-element blocks of [64 rows][128 B]
constexpr int kPBytes = kBM * kBN * 2;         // 16 KB: one block of [128 rows][128 B]
constexpr int kSmemBytes = kQBytes + 4 * kTileBytes + kPBytes + 64 /*barrier, tmem base, flag*/;
constexpr uint32_t kTmemCols = 256;            // S: columns [0,64), O: columns [128,256)
constexpr uint32_t kTmemO = 128;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;      // in log2 units: P stays below 2^8
constexpr uint32_t kSpinLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
// Bounded wait on an mbarrier phase; returns false on timeout.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
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

// Shared-memory matrix descriptor, 128-byte swizzle; strides in bytes.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3fffu);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
  d |= (uint64_t)1 << 46;     // descriptor version of this architecture
  d |= (uint64_t)2 << 61;     // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, A K-major, B K-major or MN-major.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,"
      "%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,"
      "%30,%31,%32};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
        "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
        "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])),
        "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])), "r"(__float_as_uint(v[16])),
        "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
        "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])),
        "r"(__float_as_uint(v[23])), "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])),
        "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])), "r"(__float_as_uint(v[28])),
        "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// Byte offset inside a [rows][128 B] block with the 128-byte swizzle: 16-byte chunk c of row r.
__device__ __forceinline__ uint32_t blk_off(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

}  // namespace tc

__global__ void __launch_bounds__(tc::kThreads, 2)
attn_tc_kernel(const __nv_bfloat16* __restrict__ Kc, const __nv_bfloat16* __restrict__ Vc,
               const int32_t* __restrict__ cache_len, const __nv_bfloat16* __restrict__ Q,
               __nv_bfloat16* __restrict__ O, float* __restrict__ lse, float* __restrict__ part_o,
               float2* __restrict__ part_ml, int Hq, int Hkv, int T_q, int capacity, int appended, float scale,
               int n_splits, int row_tiles, int* __restrict__ d_status) {
  using namespace tc;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);                          // tiles need 1024-byte alignment (checked below)
  const uint32_t sQ = base;
  const uint32_t sK = sQ + kQBytes;            // 2 stages
  const uint32_t sV = sK + 2 * kTileBytes;     // 2 stages
  const uint32_t sP = sV + 2 * kTileBytes;
  const uint32_t sBar = sP + kPBytes;          // mbarrier (8 B), tmem base (4 B), failure flag (4 B)
  unsigned char* gen_base = smem_raw;
  if ((base & 1023u) != 0) {                                         // never expected; refuse rather than compute garbage
    if (threadIdx.x == 0) atomicMax(d_status, (int)CHECK_SMEM_ALIGNMENT);
    return;
  }
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(gen_base + kQBytes + 4 * kTileBytes + kPBytes + 8);
  volatile uint32_t* s_fail = s_tmem + 1;

  const int tid = threadIdx.x, warp = tid >> 5;
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
  const int cta_visible = len + (n_app ? last_row / G + 1 : 0);
  const int n_tiles = (total + kBN - 1) / kBN;
  const int tps = (n_tiles + n_splits - 1) / n_splits;
  const int tile0 = split * tps;
  const int tile1 = min(min(tile0 + tps, n_tiles), (cta_visible + kBN - 1) / kBN);

  // ---- set-up: barrier, tensor memory ----
  if (tid == 0) {
    mbar_init(sBar, 1);
    *s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sBar + 8), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);   // this warp's 32 lanes

  // ---- stage Q and the first K/V tile ----
  const int my_row = row_base + tid;                    // this thread's packed row
  for (int i = tid; i < kBM * 16; i += kThreads) {
    const int r = i >> 4, c = i & 15;
    const int rr = row_base + r;
    const bool ok = rr < rows_total;
    const int t = ok ? rr / G : 0, g = ok ? rr % G : 0;
    const __nv_bfloat16* src = Q + (((size_t)b * T_q + t) * Hq + h * G + g) * kD + c * 8;
    cp_async16(sQ + (c >> 3) * (kBM * 128) + blk_off(r, c & 7), src, ok);
  }
  const __nv_bfloat16* kbase = Kc + (size_t)bh * capacity * kD;
  const __nv_bfloat16* vbase = Vc + (size_t)bh * capacity * kD;
  // K and V tiles live in separate 2-stage rings so that K can be fetched one tile further ahead than V.
  auto load_kv = [&](const __nv_bfloat16* gbase, uint32_t sbase, int tile, int stage) {
    const int j0 = tile * kBN;
    for (int i = tid; i < kBN * 16; i += kThreads) {
      const int r = i >> 4, c = i & 15;
      const bool ok = j0 + r < total;
      const size_t off = (size_t)(ok ? j0 + r : 0) * kD + c * 8;
      cp_async16(sbase + stage * kTileBytes + (c >> 3) * (kBN * 128) + blk_off(r, c & 7), gbase + off, ok);
    }
  };
  const bool have_work = tile0 < tile1;
  if (have_work) {
    load_kv(kbase, sK, tile0, 0);
    load_kv(vbase, sV, tile0, 0);
  }
  cp_async_commit();
  if (tile0 + 1 < tile1) load_kv(kbase, sK, tile0 + 1, 1);
  cp_async_commit();

  constexpr uint32_t kIdescS = instr_desc(kBM, kBN, false);
  constexpr uint32_t kIdescO = instr_desc(kBM, kD, true);
  auto issue_s = [&](int stage) {      // S = Q K^T, 8 k-steps of 16 over the two 64-element blocks
#pragma unroll
    for (int ks = 0; ks < kD / 16; ++ks) {
      const uint32_t koff = (ks >> 2) * (kBM * 128) + (ks & 3) * 32;
      const uint32_t boff = (ks >> 2) * (kBN * 128) + (ks & 3) * 32;
      mma_f16(tmem, smem_desc(sQ + koff, 16, 1024), smem_desc(sK + stage * kTileBytes + boff, 16, 1024), kIdescS,
              ks > 0);
    }
  };
  auto issue_o = [&](int stage, uint32_t accumulate) {   // O += P V, 4 k-steps of 16 slots
#pragma unroll
    for (int ks = 0; ks < kBN / 16; ++ks) {
      mma_f16(tmem + kTmemO, smem_desc(sP + ks * 32, 16, 1024),
              smem_desc(sV + stage * kTileBytes + ks * 16 * 128, kBN * 128, 1024), kIdescO, accumulate | (ks > 0));
    }
  };

  cp_async_wait<1>();      // Q, K and V of the first tile (the second K tile may still be in flight)
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  if (have_work && tid == 0) {
    tc_fence_after();
    issue_s(0);
    mma_commit(sBar);
  }

  const int vis = len + (n_app ? min(my_row, rows_total - 1) / G + 1 : 0);
  const float sl2 = scale * kLog2e;
  float m = -INFINITY, l = 0.f;
  uint32_t phase = 0;
  bool failed = false;

  for (int tile = tile0; tile < tile1; ++tile) {
    const int it = tile - tile0;
    const int stage = it & 1;
    // S of this tile is ready and every earlier MMA (hence the previous P V) has completed
    if (!failed && !mbar_wait(sBar, phase)) { failed = true; *s_fail = 1; }
    failed = __any_sync(0xffffffffu, failed);
    phase ^= 1;
    tc_fence_after();
    // K of this tile and V of the previous one are no longer in use: refill those stages now, a full
    // iteration before the data is needed
    if (tile + 2 < tile1) load_kv(kbase, sK, tile + 2, stage);
    if (tile + 1 < tile1) load_kv(vbase, sV, tile + 1, stage ^ 1);
    cp_async_commit();

    // ---- softmax of this thread's row ----
    float s[kBN];
    tmem_ld32(lane_addr, s);
    tmem_ld32(lane_addr + 32, s + 32);
    const int j0 = tile * kBN;
    if (j0 + kBN > vis) {        // only tiles that reach past this row's visible range need the mask
#pragma unroll
      for (int j = 0; j < kBN; ++j)
        if (j0 + j >= vis) s[j] = -INFINITY;
    }
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < kBN; ++j) mx = fmaxf(mx, s[j]);
    const float m_cand = fmaxf(m, mx * sl2);
    // keep the old reference maximum unless it would let P exceed 2^8 (or nothing has been seen yet)
    const bool grow = (m_cand - m > kRescaleThreshold) || (m == -INFINITY && m_cand > -INFINITY);
    const float m_use = grow ? m_cand : m;
    const float mu = (m_use == -INFINITY) ? 0.f : m_use;
    float psum = 0.f;
    uint32_t pk[kBN / 2];
#pragma unroll
    for (int j = 0; j < kBN; j += 2) {
      const float p0 = fast_exp2(fmaf(s[j], sl2, -mu));
      const float p1 = fast_exp2(fmaf(s[j + 1], sl2, -mu));
      psum += p0 + p1;
      pk[j >> 1] = pack_bf16(p0, p1);
    }
    const float corr = grow ? fast_exp2(m - mu) : 1.0f;      // exp2(-inf) = 0 on the first tile
    l = l * corr + psum;
    m = m_use;
    // P row -> shared memory (K-major block, 8 chunks of 8 slots)
#pragma unroll
    for (int c = 0; c < kBN / 8; ++c) {
      asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(sP + blk_off(tid, c)), "r"(pk[c * 4]),
                   "r"(pk[c * 4 + 1]), "r"(pk[c * 4 + 2]), "r"(pk[c * 4 + 3]) : "memory");
    }
    // rescale O in tensor memory when some row of this warp moved its maximum
    if (it > 0 && __any_sync(0xffffffffu, grow)) {
#pragma unroll 1
      for (int c0 = 0; c0 < kD; c0 += 32) {
        float o[32];
        tmem_ld32(lane_addr + kTmemO + c0, o);
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] *= corr;
        tmem_st32(lane_addr + kTmemO + c0, o);
      }
      tmem_wait_st();
    }
    cp_async_wait<1>();          // everything but this iteration's prefetch has landed: V of this tile, K of the next
    fence_proxy_async();         // P (st.shared) and K/V (cp.async) become visible to the tensor core
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && !*s_fail) {
      tc_fence_after();
      issue_o(stage, it > 0);
      if (tile + 1 < tile1) issue_s(stage ^ 1);
      mma_commit(sBar);
    }
  }
  cp_async_wait<0>();
  if (have_work) {               // the last P V
    if (!failed && !mbar_wait(sBar, phase)) { failed = true; *s_fail = 1; }
    failed = __any_sync(0xffffffffu, failed);
    tc_fence_after();
  }

  // ---- write this thread's row (tensor-memory loads are warp-wide, stores are per row) ----
  {
    const bool store = my_row < rows_total && !failed;
    const int rr = min(my_row, rows_total - 1);
    const int t = rr / G, hq = h * G + rr % G;
    const size_t orow = ((size_t)b * T_q + t) * Hq + hq;
    const float inv = (n_splits == 1) ? (l > 0.f ? 1.0f / l : 0.f) : 1.0f;
#pragma unroll 1
    for (int c0 = 0; c0 < kD; c0 += 32) {
      float o[32];
      if (have_work) {
        tmem_ld32(lane_addr + kTmemO + c0, o);
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = 0.f;
      }
      if (!store) continue;
      if (n_splits == 1) {
        __nv_bfloat16* op = O + orow * kD + c0;
#pragma unroll
        for (int i = 0; i < 32; i += 8) {
          uint4 v;
          v.x = pack_bf16(o[i] * inv, o[i + 1] * inv);
          v.y = pack_bf16(o[i + 2] * inv, o[i + 3] * inv);
          v.z = pack_bf16(o[i + 4] * inv, o[i + 5] * inv);
          v.w = pack_bf16(o[i + 6] * inv, o[i + 7] * inv);
          *reinterpret_cast<uint4*>(op + i) = v;
        }
      } else {
        float* po = part_o + (orow * n_splits + split) * kD + c0;
#pragma unroll
        for (int i = 0; i < 32; i += 4) *reinterpret_cast<float4*>(po + i) = make_float4(o[i], o[i + 1], o[i + 2], o[i + 3]);
      }
    }
    if (store) {
      if (n_splits == 1) {
        if (lse != nullptr) lse[((size_t)b * Hq + hq) * T_q + t] = l > 0.f ? m * kLn2 + logf(l) : -INFINITY;
      } else {
        part_ml[orow * n_splits + split] = make_float2(l > 0.f ? m * kLn2 : -INFINITY, l);
      }
    }
  }
  if (failed && tid == 0) atomicMax(d_status, (int)CHECK_WAIT_TIMEOUT);

  // ---- release tensor memory ----
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

cudaError_t launch_attn_tc(const samkv_shape_t& s, const void* Kc, const void* Vc, int capacity,
                           const int32_t* cache_len, const void* Q, int T_q, int appended, float scale, void* O,
                           float* lse, float* part_o, float2* part_ml, const AttnPlan& plan, int* d_status,
                           cudaStream_t stream) {
  const int G = s.n_q_heads / s.n_kv_heads;
  const int rows = T_q * G;
  const int row_tiles = (rows + tc::kBM - 1) / tc::kBM;
  const long long blocks = (long long)s.batch * s.n_kv_heads * row_tiles * plan.n_splits;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes);
  if (e != cudaSuccess) return e;
  attn_tc_kernel<<<(unsigned)blocks, tc::kThreads, tc::kSmemBytes, stream>>>(
      (const __nv_bfloat16*)Kc, (const __nv_bfloat16*)Vc, cache_len, (const __nv_bfloat16*)Q, (__nv_bfloat16*)O, lse,
      part_o, part_ml, s.n_q_heads, s.n_kv_heads, T_q, capacity, appended, scale, plan.n_splits, row_tiles, d_status);
  return cudaGetLastError();
}

}  // namespace samkv
