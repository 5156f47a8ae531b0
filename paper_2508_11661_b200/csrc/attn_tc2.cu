// Warp-specialised tcgen05 attention over the compact cache for prefill chunks (Sec. 3.3), d = 128.
//
// One CTA per SM: two 128-row query tiles (256 packed rows of one (batch, kv head); row r = token r / G,
// group member r % G) and one KV split, walked in tiles of 128 slots.  Roles:
//   warps 0-3   softmax of query tile 0: thread t owns row t; it reads its S row from tensor memory twice
//               (maximum, then exponentials), writes P as packed bf16 back into tensor memory over the S
//               columns it has consumed, and rescales O there only when its reference maximum grew by
//               more than 2^8; at the end it writes the row out
//   warps 4-7   the same for query tile 1
//   warp  8     one thread issues every tcgen05.mma: S_q = Q_q K^T (operands in shared memory, M=128 N=128
//               K=16 x 8) and O_q += P_q V (P from tensor memory, V as the MN-major B operand in its natural
//               [slot][d] layout, K=16 x 8); while one query tile exponentiates, the tensor pipe works on the other
//   warp  9     loader: K and V tiles arrive by TMA (cp.async.bulk.tensor, 128-byte swizzle) in two 2-stage rings
// Taking P from tensor memory halves the tensor core's shared-memory operand traffic, which otherwise
// saturates the shared-memory pipeline (an M128 N128 K16 product with both operands in shared memory
// reads 128 B per cycle) and slows every barrier poll and store of the other warps.
// Tensor memory: S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P_q overlays the first 64 columns of S_q.
// All hand-offs are mbarriers polled by one lane per warp; every wait is bounded and a timeout is recorded
// as a device check, after which the CTA drains and frees its tensor memory.  The TMA loads read this
// GPU's memory only and use no multicast.
#include "tc_common.cuh"

namespace samkv {
namespace tc2 {
using namespace tc;

constexpr int kBM = 128, kBN = 128, kD = 128;
constexpr int kStages = 2;                    // K and V each have their own 2-stage ring
constexpr int kSoftmaxWarps = 8;              // 4 per query tile: thread t of a tile owns row t
constexpr int kMmaWarp = 8, kLoadWarp = 9;
constexpr int kThreads = 320;                 // 8 softmax warps + MMA warp + loader warp
constexpr int kQBytes = kBM * kD * 2;         // 32 KB per query tile
constexpr int kTileBytes = kBN * kD * 2;      // 32 KB per K or V tile
constexpr int kOffQ = 0;
constexpr int kOffK = 2 * kQBytes;
constexpr int kOffV = kOffK + kStages * kTileBytes;
constexpr int kOffBar = kOffV + kStages * kTileBytes;
constexpr int kSmemBytes = kOffBar + 256;
constexpr uint32_t kTmemCols = 512;           // S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P_q overlays S_q
constexpr uint32_t kTmemO = 256;

// barrier slots (8 bytes each) inside the barrier block
enum Bar { K_FULL = 0, K_EMPTY = 2, V_FULL = 4, V_EMPTY = 6, KV_TMA = 8, S_FULL = 9, P_READY = 11, O_FINAL = 13, Q_READY = 14, N_BARS = 15 };


}  // namespace tc2

__global__ void __launch_bounds__(tc2::kThreads, 1)
attn_tc2_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                const int32_t* __restrict__ cache_len, const __nv_bfloat16* __restrict__ Q,
                __nv_bfloat16* __restrict__ O, float* __restrict__ lse, float* __restrict__ part_o,
                float2* __restrict__ part_ml, int Hq, int Hkv, int T_q, int capacity, int appended, float scale,
                int n_splits, int row_tiles, int* __restrict__ d_status) {
  using namespace tc2;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  if ((base & 1023u) != 0) {
    if (threadIdx.x == 0) atomicMax(d_status, (int)CHECK_SMEM_ALIGNMENT);
    return;
  }
  const uint32_t sQ = base + kOffQ, sK = base + kOffK, sV = base + kOffV, sBar = base + kOffBar;
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem_raw + kOffBar + N_BARS * 8);
  volatile uint32_t* s_fail = s_tmem + 1;
  auto bar = [&](int slot) { return sBar + 8u * slot; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = Hq / Hkv;
  const int split = blockIdx.x % n_splits;
  const int rtile = (blockIdx.x / n_splits) % row_tiles;     // pair of 128-row tiles
  const int bh = blockIdx.x / (n_splits * row_tiles);
  const int h = bh % Hkv, b = bh / Hkv;
  const int rows_total = T_q * G;
  const int row_base = rtile * 2 * kBM;
  const int n_q = (rows_total - row_base > kBM) ? 2 : 1;      // query tiles that hold real rows

  // ---- set-up ----
  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(bar(K_FULL + i), 1); mbar_init(bar(K_EMPTY + i), 1);
      mbar_init(bar(V_FULL + i), 1); mbar_init(bar(V_EMPTY + i), 1);
    }
    mbar_init(bar(KV_TMA), 1);
    mbar_init(bar(O_FINAL), 1);
    mbar_init(bar(Q_READY), kSoftmaxWarps);
    for (int q = 0; q < 2; ++q) {
      mbar_init(bar(S_FULL + q), 1);
      mbar_init(bar(P_READY + q), 4);     // one arrival per softmax warp of the tile
    }
    *s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sBar + N_BARS * 8), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();            // barriers initialised, tensor memory allocated: the roles part ways here
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  // Everything above needs nothing from the kernels before this one in the stream (they may still be running when
  // this kernel was launched as a programmatic dependent); everything below does: Q, cache_len, the appended rows and
  // the partial-result scratch.
  pdl_wait();
  int len = cache_len[b];     // (issued first: its latency overlaps the Q copies below)

  // Q tiles: cp.async by the softmax warps (rows beyond the chunk zero-filled); the MMA thread waits for Q_READY
  // before its first product
  if (warp < kSoftmaxWarps) {
    for (int i = tid; i < 2 * kBM * 16; i += kSoftmaxWarps * 32) {
      const int r = i >> 4, c = i & 15;                       // r in [0, 256)
      const int rr = row_base + r;
      const bool ok = rr < rows_total;
      const int t = ok ? rr / G : 0, g = ok ? rr % G : 0;
      const __nv_bfloat16* src = Q + (((size_t)b * T_q + t) * Hq + h * G + g) * kD + c * 8;
      cp_async16(sQ + (r >> 7) * kQBytes + (c >> 3) * (kBM * 128) + blk_off(r & 127, c & 7), src, ok);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  }

  len = max(0, min(len, capacity));
  const int n_app = (appended && len + T_q <= capacity) ? T_q : 0;
  const int total = len + n_app;
  const int last_row = min(row_base + 2 * kBM, rows_total) - 1;
  const int cta_visible = len + (n_app ? last_row / G + 1 : 0);
  const int n_tiles = (total + kBN - 1) / kBN;
  const int tps = (n_tiles + n_splits - 1) / n_splits;
  const int tile0 = split * tps;
  const int tile1 = min(min(tile0 + tps, n_tiles), (cta_visible + kBN - 1) / kBN);
  const int nt = max(tile1 - tile0, 0);

  if (warp < kSoftmaxWarps) {
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    fence_proxy_async();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar(Q_READY));
  }

  if (warp == kLoadWarp) {
    // ================= loader: K ring and V ring =================
    for (int j = 0; j < nt; ++j) {
      const int s = j % kStages;
      const uint32_t round = (uint32_t)(j / kStages);
      const int j0 = (tile0 + j) * kBN;
      mbar_wait_warp(bar(K_EMPTY + s), (round & 1) ^ 1, s_fail);
      if (lane == 0) {
        mbar_expect_tx(bar(K_FULL + s), kTileBytes);
        tma_load_3d(sK + s * kTileBytes, &tmK, 0, j0, bh, bar(K_FULL + s));
        tma_load_3d(sK + s * kTileBytes + kBN * 128, &tmK, 64, j0, bh, bar(K_FULL + s));
      }
      mbar_wait_warp(bar(V_EMPTY + s), (round & 1) ^ 1, s_fail);
      const bool partial = j0 + kBN > total;                   // V rows past `total` must read as zero
      const uint32_t target = partial ? bar(KV_TMA) : bar(V_FULL + s);
      if (lane == 0) {
        mbar_expect_tx(target, kTileBytes);
        tma_load_3d(sV + s * kTileBytes, &tmV, 0, j0, bh, target);
        tma_load_3d(sV + s * kTileBytes + kBN * 128, &tmV, 64, j0, bh, target);
      }
      if (partial) {                                            // at most once per CTA: the last tile of the cache
        mbar_wait_warp(bar(KV_TMA), 0, s_fail);
        const int first_bad = total - j0;
        for (int i = lane; i < (kBN - first_bad) * 16; i += 32) {
          const int r = first_bad + (i >> 4), c = i & 15;
          asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(sV + s * kTileBytes + (c >> 3) * (kBN * 128) +
                                                                      blk_off(r, c & 7)), "r"(0) : "memory");
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(V_FULL + s));
      }
      __syncwarp();
    }
  } else if (warp == kMmaWarp) {
    // ================= MMA issuer =================
    if (lane == 0 && nt > 0) {
      constexpr uint32_t kIdescS = instr_desc(kBM, kBN, false);
      constexpr uint32_t kIdescO = instr_desc(kBM, kD, true);
      // Descriptors are built once; per instruction only the 14-bit start-address field (16-byte units) moves.
      // Building one from scratch costs tens of dependent ALU instructions on this single thread, more than
      // the 64 cycles an M128 N128 K16 product takes.
      const uint64_t dQ = smem_desc(sQ, 16, 1024), dK = smem_desc(sK, 16, 1024);
      const uint64_t dV = smem_desc(sV, kBN * 128, 1024);
      auto issue_s = [&](int q, int s) {                       // S_q = Q_q K^T : 8 k-steps over d
        const uint64_t a0 = dQ + (uint64_t)(q * (kQBytes >> 4)), b0 = dK + (uint64_t)(s * (kTileBytes >> 4));
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
          const uint32_t aoff = ((ks >> 2) * (kBM * 128) + (ks & 3) * 32) >> 4;
          const uint32_t boff = ((ks >> 2) * (kBN * 128) + (ks & 3) * 32) >> 4;
          mma_ss(tmem + q * kBN, a0 + aoff, b0 + boff, kIdescS, ks > 0);
        }
        mma_commit(bar(S_FULL + q));
      };
      auto issue_pv = [&](int q, int s, uint32_t accumulate) { // O_q += P_q V : 8 k-steps over the 128 slots, P from tensor memory
        const uint64_t b0 = dV + (uint64_t)(s * (kTileBytes >> 4));
#pragma unroll
        for (int ks = 0; ks < kBN / 16; ++ks)
          mma_ts(tmem + kTmemO + q * kD, tmem + q * kBN + ks * 8, b0 + ((ks * 16 * 128) >> 4), kIdescO,
                 accumulate | (ks > 0));
      };
      mbar_wait(bar(Q_READY), 0, s_fail);
      mbar_wait(bar(K_FULL + 0), 0, s_fail);
      tc_fence_after();
      for (int q = 0; q < n_q; ++q) issue_s(q, 0);
      mma_commit(bar(K_EMPTY + 0));
      for (int j = 0; j < nt; ++j) {
        const int s = j % kStages, s1 = (j + 1) % kStages;
        mbar_wait(bar(V_FULL + s), (uint32_t)((j / kStages) & 1), s_fail);
        if (j + 1 < nt) mbar_wait(bar(K_FULL + s1), (uint32_t)(((j + 1) / kStages) & 1), s_fail);
        for (int q = 0; q < n_q; ++q) {
          // P_q of this tile is in tensor memory (and S_q has been consumed): O_q += P_q V, then S_q of the
          // next tile may overwrite the same columns (the tensor pipe executes in issue order)
          mbar_wait(bar(P_READY + q), (uint32_t)(j & 1), s_fail);
          tc_fence_after();
          issue_pv(q, s, j > 0);
          if (j + 1 < nt) issue_s(q, s1);
        }
        mma_commit(bar(V_EMPTY + s));                            // every MMA so far finished: V_j (and K_{j+1}) are free
        if (j + 1 < nt) mma_commit(bar(K_EMPTY + s1));
      }
      mma_commit(bar(O_FINAL));
    }
  } else {
    // ================= softmax warps =================
    const int q = warp >> 2;                                    // query tile of this warp
    const int wl = warp & 3;                                    // tensor-memory lane quarter
    const int row_in_tile = wl * 32 + lane;
    const int my_row = row_base + q * kBM + row_in_tile;
    const uint32_t lane_addr = tmem + ((uint32_t)(wl * 32) << 16);
    const uint32_t tS = lane_addr + q * kBN, tO = lane_addr + kTmemO + q * kD;
    const bool active = q < n_q;                                // a tile without real rows idles
    const int vis = len + (n_app ? min(my_row, rows_total - 1) / G + 1 : 0);
    const float sl2 = scale * kLog2e;
    float m = -INFINITY, l = 0.f;

    if (active) {
      for (int j = 0; j < nt; ++j) {
        // S_q(j) complete; so is every earlier MMA, in particular P_q(j-1) V, hence O_q and the P columns are ours
        mbar_wait_warp(bar(S_FULL + q), (uint32_t)(j & 1), s_fail);
        tc_fence_after();
        const int j0 = (tile0 + j) * kBN;
        const bool masked = j0 + kBN > vis;
        // pass 1: row maximum (two loads in flight)
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll 1
        for (int c0 = 0; c0 < kBN; c0 += 64) {
          float sv[64];
          tmem_ld32_nowait(tS + c0, sv);
          tmem_ld32_nowait(tS + c0 + 32, sv + 32);
          tmem_wait_ld();
          if (masked) {
#pragma unroll
            for (int i = 0; i < 64; ++i)
              if (j0 + c0 + i >= vis) sv[i] = -INFINITY;
          }
#pragma unroll
          for (int i = 0; i < 64; i += 4) {
            mx0 = fmaxf(mx0, sv[i]); mx1 = fmaxf(mx1, sv[i + 1]); mx2 = fmaxf(mx2, sv[i + 2]); mx3 = fmaxf(mx3, sv[i + 3]);
          }
        }
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
        const float m_cand = fmaxf(m, mx * sl2);
        const bool grow = (m_cand - m > kRescaleThreshold) || (m == -INFINITY && m_cand > -INFINITY);
        const float m_use = grow ? m_cand : m;
        const float mu = (m_use == -INFINITY) ? 0.f : m_use;
        const float corr = grow ? fast_exp2(m - mu) : 1.0f;
        // rescale O in tensor memory when some row of this warp moved its reference maximum
        if (j > 0 && __any_sync(0xffffffffu, grow)) {
#pragma unroll 1
          for (int c0 = 0; c0 < kD; c0 += 32) {
            float o[32];
            tmem_ld32(tO + c0, o);
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] *= corr;
            tmem_st32(tO + c0, o);
          }
        }
        // pass 2: P = exp2(S * scale - m), rounded to bf16, written over the S columns already consumed
        float ps0 = 0.f, ps1 = 0.f, ps2 = 0.f, ps3 = 0.f;
#pragma unroll 1
        for (int c0 = 0; c0 < kBN; c0 += 32) {
          float sv[32];
          tmem_ld32(tS + c0, sv);
          if (masked) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (j0 + c0 + i >= vis) sv[i] = -INFINITY;
          }
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            const float p0 = fast_exp2(fmaf(sv[i], sl2, -mu));
            const float p1 = fast_exp2(fmaf(sv[i + 1], sl2, -mu));
            const float p2 = fast_exp2(fmaf(sv[i + 2], sl2, -mu));
            const float p3 = fast_exp2(fmaf(sv[i + 3], sl2, -mu));
            ps0 += p0; ps1 += p1; ps2 += p2; ps3 += p3;
            pk[i >> 1] = pack_bf16(p0, p1);
            pk[(i >> 1) + 1] = pack_bf16(p2, p3);
          }
          tmem_st16(tS + (c0 >> 1), pk);
        }
        l = l * corr + ((ps0 + ps1) + (ps2 + ps3));
        m = m_use;
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(P_READY + q));
      }
      if (nt > 0) {
        mbar_wait_warp(bar(O_FINAL), 0, s_fail);
        tc_fence_after();
      }
      // ---- write this thread's row ----
      const bool failed = *s_fail != 0;
      const bool store = my_row < rows_total && !failed;
      const int rr = min(my_row, rows_total - 1);
      const int t = rr / G, hq = h * G + rr % G;
      const size_t orow = ((size_t)b * T_q + t) * Hq + hq;
      const float inv = (n_splits == 1) ? (l > 0.f ? 1.0f / l : 0.f) : 1.0f;
#pragma unroll 1
      for (int c0 = 0; c0 < kD; c0 += 32) {
        float o[32];
        if (nt > 0) {
          tmem_ld32(tO + c0, o);
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
          for (int i = 0; i < 32; i += 4)
            *reinterpret_cast<float4*>(po + i) = make_float4(o[i], o[i + 1], o[i + 2], o[i + 3]);
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
  }

  // ---- teardown: every role arrives here, then the allocating warp frees tensor memory ----
  tc_fence_before();
  __syncthreads();
  pdl_launch_dependents();      // results are written: the merge kernel may be scheduled (it still waits for our exit)
  if (tid == 0 && *s_fail) atomicMax(d_status, (int)CHECK_WAIT_TIMEOUT);
  if (warp == kMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------
// Host side: tensor maps for the K and V slabs of one layer (tc_common.cuh), then the launch.
// ---------------------------------------------------------------------------------------------
cudaError_t launch_attn_tc2(const samkv_shape_t& s, const void* Kc, const void* Vc, int capacity,
                            const int32_t* cache_len, const void* Q, int T_q, int appended, float scale, void* O,
                            float* lse, float* part_o, float2* part_ml, const AttnPlan& plan, int* d_status,
                            cudaStream_t stream) {
  const int G = s.n_q_heads / s.n_kv_heads;
  const int rows = T_q * G;
  const int row_tiles = (rows + 2 * tc2::kBM - 1) / (2 * tc2::kBM);
  const long long blocks = (long long)s.batch * s.n_kv_heads * row_tiles * plan.n_splits;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  CUtensorMap tmK, tmV;
  if (!tc::make_kv_map(&tmK, Kc, capacity, s.batch * s.n_kv_heads) ||
      !tc::make_kv_map(&tmV, Vc, capacity, s.batch * s.n_kv_heads))
    return cudaErrorInvalidValue;
  cudaError_t e = ensure_dynamic_smem<3>(attn_tc2_kernel, tc2::kSmemBytes);
  if (e != cudaSuccess) return e;
  // Launched so that it may start while the kernel before it in the stream (the append of the chunk) is still
  // running: set-up and the Q loads need nothing from it; the loader waits before its first K/V tile.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)blocks);
  cfg.blockDim = dim3(tc2::kThreads);
  cfg.dynamicSmemBytes = tc2::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, attn_tc2_kernel, tmK, tmV, cache_len, (const __nv_bfloat16*)Q, (__nv_bfloat16*)O, lse,
                            part_o, part_ml, s.n_q_heads, s.n_kv_heads, T_q, capacity, appended, scale, plan.n_splits,
                            row_tiles, d_status);
}

}  // namespace samkv
