// Warp-specialised tcgen05 attention over the compact cache for prefill chunks (Sec. 3.3), d = 128.
//
// One CTA per SM: one 128-row query tile (packed rows of one (batch, kv head); row r = token r / G, group member
// r % G) and one KV range, walked in tiles of 128 slots.  The tiles of the range are dealt to two independent groups,
// even tiles to group 0 and odd tiles to group 1; each group keeps its own running maximum, denominator and output
// accumulator, and the two partial results are merged at the end like two KV splits.  While one group exponentiates,
// the tensor pipe works on the other group's products.  Roles:
//   warps 0-3   softmax of group 0: thread t owns row t (no exchange between threads).  It takes its whole S row from
//   warps 4-7   tensor memory into registers (maximum, then exponentials), writes P as packed bf16 back over the first
//   (group 1)   half of the S columns, and rescales O there only when its reference maximum grew by more than 2^64
//               (P may exceed 1: bf16 has the exponent range of fp32, and l and O keep a margin of 2^63 for their sums).
//               Scaling and row sums run as packed two-wide fp32 operations, and the bf16 rounding of P on the integer
//               pipe, which leaves the special-function unit to the exponentials.
//   warp  8/9   issuer of group 0 / 1 (one thread issues, the warp waits converged): O_g += P(t) V(t) as soon as P(t)
//               is complete and V(t) and K(t+2) have landed (one barrier collects all three), then S(t+2) = Q K(t+2)^T
//               into the buffer P(t) occupied (the tensor pipe keeps a thread's issue order), then one commit that
//               tells the softmax warps "S(t+2) ready, O at rest" and the loader "stages free".  One poll and one
//               commit per 16 products: a thread can run only about two products ahead of the pipe, and every poll or
//               commit costs it 100-300 cycles, which the other issuer's products cover.
//   warp 10     loader: K and V tiles (3 stages each) arrive by TMA (cp.async.bulk.tensor, 128-byte swizzle)
//   warp 11     idle: it completes the third warpgroup, which hands registers to the softmax warps (setmaxnreg)
// The chunk's own K/V rows (the "append" of the incremental prefill) are written into the cache by this kernel: every
// CTA whose KV range reaches past cache_len copies the rows of its (batch, kv head) itself before its loader fetches
// those tiles.  Several CTAs then write the same bytes to the same addresses, which is harmless and needs no
// dependency between CTAs.
// Tensor memory: S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P_g overlays the first 64 columns of S_g.
// Barriers are indexed by tile number mod 6 (a multiple of the group count 2 and the stage count 3), so that no
// waiter can be a whole round behind.
// With exactly two KV splits the grid is launched in clusters of two CTAs (the two splits of one query tile): the
// CTAs swap the (m, l, O) of half of the rows each through distributed shared memory between two cluster barriers and
// each writes the final result of its half; every thread of both CTAs walks through both barriers on every path.
// Every wait is bounded and a timeout is recorded as a device check, after which the CTA drains and frees its tensor
// memory.  The TMA loads read this GPU's memory only and use no multicast.  Nothing the caller may have produced just
// before the call (Q, the cache, cache_len) is read before the grid-dependency wait.
#include "tc_common.cuh"

namespace samkv {
namespace tc4 {
using namespace tc;

constexpr int kBM = 128, kBN = 128, kD = 128;
constexpr int kStages = 3;                    // K and V each have their own ring
constexpr int kParts = 2;                     // the epilogue splits a row's 128 output columns between two threads
constexpr int kPartCols = kD / kParts;        // 64
constexpr int kSoftmaxWarps = 8;              // 4 per group
constexpr int kMmaWarp0 = 8, kMmaWarp1 = 9, kLoadWarp = 10;   // warp 11 only fills up the third warpgroup
constexpr int kThreads = 12 * 32;
// Register budget: the kernel starts with 65536 / 384 = 168 registers per thread; the third warpgroup hands most of
// its share to the softmax warps, which keep a whole 128-column score row in registers.
constexpr int kRegsSoftmax = 224, kRegsOther = 56;
constexpr int kQBytes = kBM * kD * 2;         // 32 KB
constexpr int kTileBytes = kBN * kD * 2;      // 32 KB per K or V tile
constexpr int kOffQ = 0;
constexpr int kOffK = kQBytes;
constexpr int kOffV = kOffK + kStages * kTileBytes;
constexpr int kOffX = kOffV + kStages * kTileBytes;    // (m, l) of both groups per row: [2][128] float2
constexpr int kOffBar = kOffX + 2 * kBM * 8;
constexpr int kSmemBytes = kOffBar + 256;
static_assert(kSmemBytes <= 232448, "shared memory of one CTA");
// O is rescaled only when a row's reference maximum grows by more than this (log2 units).
constexpr float kGrowThreshold = 64.0f;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemO = 256;

constexpr int kTurnBar = 5;                   // named barriers 5, 6: whose turn it is to exponentiate (1-4: row pairs)
constexpr int kRound = 6;                     // barrier slots per kind: tile t uses slot t % 6, phase t / 6
enum Bar {
  GO = 0,             // O += P(t) V(t) and S(t+2) may be issued: P(t) complete (4 softmax warps), V(t) and K(t+2) landed
  FULL = kRound,      // S(t) is complete, and so is O += P(t-2) V(t-2): the group may read S(t) and touch O; K stage of
                      // tile t and V stage of tile t-2 are free
  K01 = 2 * kRound,   // K(0), K(1) have landed (two slots)
  KV_TMA = 2 * kRound + 2, O_FINAL /* two slots */, Q_READY = O_FINAL + 2,
  APPENDED,           // this CTA's copy of the chunk's K/V rows into the cache is complete (8 softmax warps)
  N_BARS
};

// two fp32 values in one 64-bit register, for the packed fp32 instructions
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
}  // namespace tc4

// kPair: the grid is launched in clusters of two CTAs, the two KV splits of one (batch, kv head, query tile).  Each
// CTA hands the (m, l, O) of half of the rows to the other through distributed shared memory and writes the final
// rows of its half: no partial results in global memory and no merge kernel.  The cache length of an appended chunk
// is then bumped by the last CTA of the grid to finish (a counter in the workspace's status block).
template <bool kPair>
__global__ void __launch_bounds__(tc4::kThreads, 1)
attn_tc4_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                int32_t* cache_len, const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ Kq,
                const __nv_bfloat16* __restrict__ Vq, __nv_bfloat16* Kc, __nv_bfloat16* Vc,
                __nv_bfloat16* __restrict__ O, float* __restrict__ lse, float* __restrict__ part_o,
                float2* __restrict__ part_ml, int Hq, int Hkv, int T_q, int capacity, float scale,
                int n_splits, int row_tiles, int* __restrict__ d_status) {
  using namespace tc4;
  const int appended = Kq != nullptr;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  // A misaligned buffer (never seen: the declaration asks for 1024 bytes) is reported and the CTA does no tile work,
  // but it still walks through every barrier below, so its cluster partner is not left waiting.
  const bool bad_smem = (base & 1023u) != 0;
  if (bad_smem && threadIdx.x == 0) atomicMax(d_status, (int)CHECK_SMEM_ALIGNMENT);
  auto pair_sync = [&]() {                                    // all threads of both CTAs of the cluster
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  };
  const uint32_t sQ = base + kOffQ, sK = base + kOffK, sV = base + kOffV, sBar = base + kOffBar;
  float2* x_ml = reinterpret_cast<float2*>(smem_raw + kOffX);         // [group][row] (m, l)
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem_raw + kOffBar + N_BARS * 8);
  volatile uint32_t* s_fail = s_tmem + 1;
  auto bar = [&](int slot) { return sBar + 8u * slot; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = Hq / Hkv;
  const int split = blockIdx.x % n_splits;
  const int rtile = (blockIdx.x / n_splits) % row_tiles;
  const int bh = blockIdx.x / (n_splits * row_tiles);
  const int h = bh % Hkv, b = bh / Hkv;
  const int rows_total = T_q * G;
  const int row_base = rtile * kBM;

  // ---- set-up: nothing here reads global memory ----
  if (tid == 0) {
    for (int i = 0; i < kRound; ++i) {
      mbar_init(bar(GO + i), 4 + 1);
      mbar_init(bar(FULL + i), 1);
    }
    mbar_init(bar(K01), 1);
    mbar_init(bar(K01 + 1), 1);
    mbar_init(bar(KV_TMA), 1);
    mbar_init(bar(O_FINAL), 1);
    mbar_init(bar(O_FINAL + 1), 1);
    mbar_init(bar(Q_READY), kSoftmaxWarps);
    mbar_init(bar(APPENDED), kSoftmaxWarps);
    *s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sBar + N_BARS * 8), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();            // barriers initialised, tensor memory allocated: the roles part ways here
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  // Everything above needs nothing from the kernels before this one in the stream (they may still be running when
  // this kernel was launched as a programmatic dependent); everything below does: Q, cache_len, the cache rows.
  pdl_wait();
  int len = cache_len[b];     // (issued first: its latency overlaps the Q copies below)

  // Q tile: cp.async by the softmax warps (rows beyond the chunk zero-filled)
  if (warp < kSoftmaxWarps) {
    for (int i = tid; i < kBM * 16; i += kSoftmaxWarps * 32) {
      const int r = i >> 4, c = i & 15;
      const int rr = row_base + r;
      const bool ok = rr < rows_total;
      const int t = ok ? rr / G : 0, g = ok ? rr % G : 0;
      const __nv_bfloat16* src = Q + (((size_t)b * T_q + t) * Hq + h * G + g) * kD + c * 8;
      cp_async16(sQ + (c >> 3) * (kBM * 128) + blk_off(r, c & 7), src, ok);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  len = max(0, min(len, capacity));
  const int n_app = (appended && len + T_q <= capacity) ? T_q : 0;
  const int total = len + n_app;
  const int last_row = min(row_base + kBM, rows_total) - 1;
  const int cta_visible = len + (n_app ? last_row / G + 1 : 0);
  const int n_tiles = (total + kBN - 1) / kBN;
  const int tps = (n_tiles + n_splits - 1) / n_splits;
  const int tile0 = split * tps;
  const int tile1 = min(min(tile0 + tps, n_tiles), (cta_visible + kBN - 1) / kBN);
  const int nt = bad_smem ? 0 : max(tile1 - tile0, 0);
  // The chunk's own K/V rows belong at slots len .. len + T_q - 1 of the cache.  Every CTA whose KV range reaches
  // past `len` writes them there itself before its loader fetches those tiles (several CTAs write the same bytes to
  // the same addresses: harmless), so no separate kernel and no dependency between CTAs is needed.  The CTA of the
  // last row tile and last split always does, so the rows are in the cache when the call completes.
  const bool copies_chunk = n_app > 0 && ((tile0 + nt) * kBN > len || (rtile == row_tiles - 1 && split == n_splits - 1));
  if (appended && n_app == 0 && blockIdx.x == 0 && tid == 0) atomicMax(d_status, (int)CHECK_APPEND_CAPACITY);

  if (warp < kSoftmaxWarps) {
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    fence_proxy_async();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar(Q_READY));
    // (after Q has been handed over: the first products do not wait for this copy, only the last tiles do)
    if (copies_chunk) {
      for (int i0 = 0; i0 < T_q * 16; i0 += kSoftmaxWarps * 32 * 4) {      // four rows' pieces in flight per thread
        uint4 vk[4], vv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int i = i0 + u * kSoftmaxWarps * 32 + tid;
          if (i < T_q * 16) {
            const size_t src = (((size_t)b * T_q + (i >> 4)) * Hkv + h) * kD + (i & 15) * 8;
            vk[u] = ld_stream(Kq + src);
            vv[u] = ld_stream(Vq + src);
          }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int i = i0 + u * kSoftmaxWarps * 32 + tid;
          if (i < T_q * 16) {
            const size_t dst = ((size_t)bh * capacity + len + (i >> 4)) * kD + (i & 15) * 8;
            *reinterpret_cast<uint4*>(Kc + dst) = vk[u];
            *reinterpret_cast<uint4*>(Vc + dst) = vv[u];
          }
        }
      }
      asm volatile("fence.proxy.async;" ::: "memory");          // the TMA loads of this CTA must see these rows
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(APPENDED));
    }
  }

  // Waits are executed by every lane of the waiting warp (the warp stays converged; a lone polling lane with the
  // other 31 parked at a warp barrier turned out slower).
  auto wait = [&](int slot, uint32_t phase) { mbar_wait(bar(slot), phase & 1u, s_fail); };

  if (warp >= kSoftmaxWarps) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
  if (warp == kLoadWarp) {
    // ================= loader: K(0), K(1), then V(t) and K(t+2) together =================
    auto load_tile = [&](const CUtensorMap* map, uint32_t dst, int t, uint32_t target) {
      const int j0 = (tile0 + t) * kBN;
      tma_load_3d(dst, map, 0, j0, bh, target);
      tma_load_3d(dst + kBN * 128, map, 64, j0, bh, target);
    };
    bool chunk_in_cache = !copies_chunk;
    auto before_tile = [&](int t) {                               // a tile that reaches past `len` holds rows of the chunk
      if (!chunk_in_cache && (tile0 + t) * kBN + kBN > len) {
        wait(APPENDED, 0);
        chunk_in_cache = true;
      }
    };
    for (int t = 0; t < 2 && t < nt; ++t) {
      before_tile(t);
      if (lane == 0) {
        mbar_expect_tx(bar(K01 + t), kTileBytes);
        load_tile(&tmK, sK + t * kTileBytes, t, bar(K01 + t));
      }
    }
    __syncwarp();
    for (int t = 0; t < nt; ++t) {
      // V(t) goes where V(t-3) was and K(t+2) where K(t-1) was: free once O += P(t-3) V(t-3) and S(t-1) have run
      if (t >= 1) wait(FULL + (t - 1) % kRound, (uint32_t)((t - 1) / kRound));
      const uint32_t sv = sV + (t % kStages) * kTileBytes;
      const bool with_k = t + 2 < nt;
      before_tile(with_k ? t + 2 : t);
      const bool partial = (tile0 + t) * kBN + kBN > total;      // V rows past `total` must read as zero
      if (lane == 0) {
        const uint32_t target = partial ? bar(KV_TMA) : bar(GO + t % kRound);
        mbar_expect_tx(target, with_k ? 2 * kTileBytes : kTileBytes);
        load_tile(&tmV, sv, t, target);
        if (with_k) load_tile(&tmK, sK + ((t + 2) % kStages) * kTileBytes, t + 2, target);   // (never with a partial tile)
      }
      if (partial) {                                              // at most once per CTA: the last tile of the cache
        wait(KV_TMA, 0);
        const int first_bad = total - (tile0 + t) * kBN;
        for (int i = lane; i < (kBN - first_bad) * 16; i += 32) {
          const int r = first_bad + (i >> 4), c = i & 15;
          asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(sv + (c >> 3) * (kBN * 128) + blk_off(r, c & 7)), "r"(0)
                       : "memory");
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(GO + t % kRound));
      }
      __syncwarp();
    }
    if constexpr (kPair) { pair_sync(); pair_sync(); }
  } else if (warp > kLoadWarp) {
    if constexpr (kPair) { pair_sync(); pair_sync(); }
  } else if (warp == kMmaWarp0 || warp == kMmaWarp1) {
    // ================= issuer of one group's products =================
    const int g = warp - kMmaWarp0;
    if (g < nt) {
      constexpr uint32_t kIdescS = instr_desc(kBM, kBN, false);
      constexpr uint32_t kIdescO = instr_desc(kBM, kD, true);
      // Descriptors are built once; per instruction only the 14-bit start-address field (16-byte units) moves.
      const uint64_t dQ = smem_desc(sQ, 16, 1024), dK = smem_desc(sK, 16, 1024);
      const uint64_t dV = smem_desc(sV, kBN * 128, 1024);
      const uint32_t tS = tmem + (uint32_t)(g * kBN), tO = tmem + kTmemO + (uint32_t)(g * kD);
      auto issue_s = [&](int t) {                               // S(t) = Q K(t)^T: 8 k-steps over d
        const uint64_t b0 = dK + (uint64_t)((t % kStages) * (kTileBytes >> 4));
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
          const uint32_t aoff = ((ks >> 2) * (kBM * 128) + (ks & 3) * 32) >> 4;
          const uint32_t boff = ((ks >> 2) * (kBN * 128) + (ks & 3) * 32) >> 4;
          mma_ss(tS, dQ + aoff, b0 + boff, kIdescS, ks > 0);
        }
      };
      wait(Q_READY, 0);
      wait(K01 + g, 0);
      tc_fence_after();
      if (lane == 0) {
        issue_s(g);
        mma_commit(bar(FULL + g));
      }
      __syncwarp();
      for (int t = g; t < nt; t += 2) {
        wait(GO + t % kRound, (uint32_t)(t / kRound));
        tc_fence_after();
        if (lane == 0) {
          const uint64_t b0 = dV + (uint64_t)((t % kStages) * (kTileBytes >> 4));
#pragma unroll
          for (int ks = 0; ks < kBN / 16; ++ks)                 // O_g += P(t) V(t): 8 k-steps over the 128 slots
            mma_ts(tO, tS + ks * 8, b0 + ((ks * 16 * 128) >> 4), kIdescO, (t >= 2) | (ks > 0));
          if (t + 2 < nt) {
            issue_s(t + 2);                                     // overwrites S(t) / P(t): the pipe keeps this thread's order
            mma_commit(bar(FULL + (t + 2) % kRound));
          } else {
            mma_commit(bar(O_FINAL + g));
          }
        }
        __syncwarp();
      }
    }
    if constexpr (kPair) { pair_sync(); pair_sync(); }
  }
  } else {
    // ================= softmax warps =================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
    const int g = warp >> 2;                                    // group: tiles t = g, g + 2, ...
    const int wl = warp & 3;                                    // tensor-memory lane quarter
    const int row_in_tile = wl * 32 + lane;
    const int my_row = row_base + row_in_tile;
    const uint32_t lane_addr = tmem + ((uint32_t)(wl * 32) << 16);
    const uint32_t tS = lane_addr + (uint32_t)(g * kBN), tOg = lane_addr + kTmemO + (uint32_t)(g * kD);
    const int vis = len + (n_app ? min(my_row, rows_total - 1) / G + 1 : 0);
    const float sl2 = scale * kLog2e;
    const uint64_t sl2_2 = pack2(sl2, sl2);
    float m = -INFINITY, l = 0.f;

    if (g == 1 && nt > 0) asm volatile("bar.arrive %0, 256;" ::"r"(kTurnBar) : "memory");   // group 0 goes first
    for (int t = g; t < nt; t += 2) {
      wait(FULL + t % kRound, (uint32_t)(t / kRound));          // S(t) complete; O_g at rest (O += P(t-2) V(t-2) has run)
      tc_fence_after();
      const int j0 = (tile0 + t) * kBN;
      const bool masked = j0 + kBN > vis;
      // the whole S row into registers (all four loads in flight), masked; row maximum over four independent chains
      float sv[kBN];
#pragma unroll
      for (int c0 = 0; c0 < kBN; c0 += 32) tmem_ld32_nowait(tS + c0, sv + c0);
      tmem_wait_ld();
      if (masked) {
#pragma unroll
        for (int i = 0; i < kBN; ++i)
          if (j0 + i >= vis) sv[i] = -INFINITY;
      }
      float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
      for (int i = 0; i < kBN; i += 8) {
        mx0 = max3(mx0, sv[i], sv[i + 1]);
        mx1 = max3(mx1, sv[i + 2], sv[i + 3]);
        mx2 = max3(mx2, sv[i + 4], sv[i + 5]);
        mx3 = max3(mx3, sv[i + 6], sv[i + 7]);
      }
      const float m_cand = fmaxf(m, fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * sl2);
      const bool grow = (m_cand - m > kGrowThreshold) || (m == -INFINITY && m_cand > -INFINITY);
      const float m_use = grow ? m_cand : m;
      const float mu = (m_use == -INFINITY) ? 0.f : m_use;
      const float corr = grow ? fast_exp2(m - mu) : 1.0f;
      // rescale O_g in tensor memory when some row of this warp moved its reference maximum (O_g is at rest)
      if (t >= 2 && __any_sync(0xffffffffu, grow)) {
#pragma unroll 1
        for (int c0 = 0; c0 < kD; c0 += 32) {
          float o[32];
          tmem_ld32(tOg + c0, o);
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] *= corr;
          tmem_st32(tOg + c0, o);
        }
      }
      // P = exp2(S * scale - m), rounded to bf16, written over the first half of the S columns (all of S sits in
      // registers by now); masked scores are -inf and give exactly 0
      const uint64_t negmu2 = pack2(-mu, -mu);
      uint64_t psa = pack2(0.f, 0.f), psb = pack2(0.f, 0.f);
      auto exps32 = [&](int c0) {
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          float x0, x1;
          unpack2(fma2(pack2(sv[c0 + 2 * i], sv[c0 + 2 * i + 1]), sl2_2, negmu2), x0, x1);
          float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
          pk[i] = round_pack_bf16(p0, p1);
          if (i & 1) psb = add2(psb, pack2(p0, p1)); else psa = add2(psa, pack2(p0, p1));
        }
        tmem_st16(tS + (c0 >> 1), pk);
      };
      // The two groups take turns on the exponentials (and with them on the special-function unit): while one
      // group exponentiates, the tensor pipe runs the other group's products.  Left alone, the groups fall into
      // step, exponentiate together and then wait for the tensor pipe together.
      asm volatile("bar.sync %0, 256;" ::"r"(kTurnBar + g) : "memory");
#pragma unroll
      for (int c0 = 0; c0 < kBN; c0 += 32) exps32(c0);
      if (t + 1 < nt) asm volatile("bar.arrive %0, 256;" ::"r"(kTurnBar + (g ^ 1)) : "memory");
      const uint64_t ps = add2(psa, psb);
      float ps0, ps1;
      unpack2(ps, ps0, ps1);
      l = l * corr + (ps0 + ps1);
      m = m_use;
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(GO + t % kRound));        // P(t) is complete
    }
    if (g < nt) {
      wait(O_FINAL + g, 0);
      tc_fence_after();
    }
    // ---- merge of the two groups: every thread needs (m, l) of both groups of its row ----
    auto row_barrier = [&]() {                                  // the two warps that share these 32 rows
      asm volatile("bar.sync %0, %1;" ::"r"(1 + wl), "n"(64) : "memory");
    };
    x_ml[g * kBM + row_in_tile] = make_float2(m, l);
    if ((g ^ 1) < nt) {                                         // the other group's accumulator is read below
      wait(O_FINAL + (g ^ 1), 0);
      tc_fence_after();
    }
    row_barrier();
    const float2 ml0 = x_ml[row_in_tile], ml1 = x_ml[kBM + row_in_tile];
    const bool hasA = ml0.y > 0.f, hasB = ml1.y > 0.f;
    m = fmaxf(hasA ? ml0.x : -INFINITY, hasB ? ml1.x : -INFINITY);
    const float wA = hasA ? fast_exp2(ml0.x - m) : 0.f, wB = hasB ? fast_exp2(ml1.x - m) : 0.f;
    const float l_row = ml0.y * wA + ml1.y * wB;
    // from here on warp w handles output columns [64 (w / 4), +64) of its rows
    const int part = warp >> 2;
    const uint32_t tO = lane_addr + kTmemO + part * kPartCols;
    auto load_o = [&](int c0, float* o) {                       // 32 merged (not yet normalised) output columns
#pragma unroll
      for (int i = 0; i < 32; ++i) o[i] = 0.f;
      // (conditions uniform over the warp: the loads are warp-wide instructions)
      if (nt > 0) {                                             // a group without tiles left its accumulator unwritten
        float a[32];
        tmem_ld32(tO + c0, a);
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = a[i] * wA;
      }
      if (nt > 1) {
        float a[32];
        tmem_ld32(tO + kD + c0, a);
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = fmaf(a[i], wB, o[i]);
      }
    };
    if constexpr (kPair) {
      // ---- merge of the two KV splits inside the cluster ----
      // Exchange area in the K ring: O parts [part][row][kPartCols] fp32 with the 16-byte chunks of a row
      // XOR-swizzled by the row (threads of a warp write different rows), then (m, l) per row.
      const uint32_t xo_local = sK + (uint32_t)((part * kBM + row_in_tile) * kPartCols * 4);
      const uint32_t xml_local = sK + (uint32_t)(kParts * kBM * kPartCols * 4 + row_in_tile * 8);
      constexpr int kChunks = kPartCols / 4;                    // 16-byte chunks per part of a row
      pair_sync();                                              // both CTAs are past their last MMA: the rings are free
      // Each CTA merges half of the rows: rows [0,64) end up in the CTA of the first split, rows [64,128) in the
      // other one, so both CTAs send 32 KB, merge 64 rows and write 16 KB instead of one of them doing it all.
      const bool mine = (row_in_tile < kBM / 2) == (split == 0);          // this CTA writes this row's result
      if (!mine) {
        uint32_t xo_remote, xml_remote;
        const uint32_t peer = (uint32_t)(split ^ 1);
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(xo_remote) : "r"(xo_local), "r"(peer));
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(xml_remote) : "r"(xml_local), "r"(peer));
#pragma unroll 1
        for (int c0 = 0; c0 < kPartCols; c0 += 32) {
          float o[32];
          load_o(c0, o);
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            const int chunk = ((c0 + i) >> 2) ^ (row_in_tile & (kChunks - 1));
            asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(xo_remote + chunk * 16), "f"(o[i]),
                         "f"(o[i + 1]), "f"(o[i + 2]), "f"(o[i + 3]) : "memory");
          }
        }
        if (part == 0)
          asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(xml_remote), "f"(m), "f"(l_row) : "memory");
      }
      pair_sync();                                              // the partner's numbers have landed
      if (mine) {
        float m1, l1;
        asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(m1), "=f"(l1) : "r"(xml_local) : "memory");
        const bool has0 = l_row > 0.f, has1 = l1 > 0.f;
        const float M = fmaxf(has0 ? m : -INFINITY, has1 ? m1 : -INFINITY);
        const float w0 = has0 ? fast_exp2(m - M) : 0.f, w1 = has1 ? fast_exp2(m1 - M) : 0.f;
        const float L = l_row * w0 + l1 * w1;
        const float inv = L > 0.f ? 1.0f / L : 0.f;
        const float a0 = w0 * inv, a1 = w1 * inv;
        const bool store = my_row < rows_total && *s_fail == 0;
        const int rr = min(my_row, rows_total - 1);
        const int t = rr / G, hq = h * G + rr % G;
        const size_t orow = ((size_t)b * T_q + t) * Hq + hq;
#pragma unroll 1
        for (int c0 = 0; c0 < kPartCols; c0 += 32) {
          float o[32];
          load_o(c0, o);
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            const int chunk = ((c0 + i) >> 2) ^ (row_in_tile & (kChunks - 1));
            float4 o1;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(o1.x), "=f"(o1.y), "=f"(o1.z), "=f"(o1.w)
                         : "r"(xo_local + chunk * 16) : "memory");
            pk[i >> 1] = pack_bf16(fmaf(o[i], a0, o1.x * a1), fmaf(o[i + 1], a0, o1.y * a1));
            pk[(i >> 1) + 1] = pack_bf16(fmaf(o[i + 2], a0, o1.z * a1), fmaf(o[i + 3], a0, o1.w * a1));
          }
          if (store) {
            __nv_bfloat16* op = O + orow * kD + part * kPartCols + c0;
#pragma unroll
            for (int i = 0; i < 16; i += 4)
              *reinterpret_cast<uint4*>(op + i * 2) = make_uint4(pk[i], pk[i + 1], pk[i + 2], pk[i + 3]);
          }
        }
        if (store && part == 0 && lse != nullptr)
          lse[((size_t)b * Hq + hq) * T_q + t] = L > 0.f ? M * kLn2 + logf(L) : -INFINITY;
      }
    } else {
      // ---- write this thread's part of the row ----
      const bool failed = *s_fail != 0;
      const bool store = my_row < rows_total && !failed;
      const int rr = min(my_row, rows_total - 1);
      const int t = rr / G, hq = h * G + rr % G;
      const size_t orow = ((size_t)b * T_q + t) * Hq + hq;
      const float inv = (n_splits == 1) ? (l_row > 0.f ? 1.0f / l_row : 0.f) : 1.0f;
#pragma unroll 1
      for (int c0 = 0; c0 < kPartCols; c0 += 32) {
        float o[32];
        load_o(c0, o);
        if (!store) continue;
        if (n_splits == 1) {
          __nv_bfloat16* op = O + orow * kD + part * kPartCols + c0;
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
          float* po = part_o + (orow * n_splits + split) * kD + part * kPartCols + c0;
#pragma unroll
          for (int i = 0; i < 32; i += 4)
            *reinterpret_cast<float4*>(po + i) = make_float4(o[i], o[i + 1], o[i + 2], o[i + 3]);
        }
      }
      if (store && part == 0) {
        if (n_splits == 1) {
          if (lse != nullptr) lse[((size_t)b * Hq + hq) * T_q + t] = l_row > 0.f ? m * kLn2 + logf(l_row) : -INFINITY;
        } else {
          part_ml[orow * n_splits + split] = make_float2(l_row > 0.f ? m * kLn2 : -INFINITY, l_row);
        }
      }
    }  // !kPair
  }

  // ---- teardown: every role arrives here, then the allocating warp frees tensor memory ----
  tc_fence_before();
  __syncthreads();
  pdl_launch_dependents();      // results are written: the merge kernel may be scheduled (it still waits for our exit)
  if (tid == 0 && *s_fail) atomicMax(d_status, (int)CHECK_WAIT_TIMEOUT);
  if constexpr (kPair) {
    // no merge kernel follows: the last CTA of the grid to get here knows that every CTA has read cache_len
    if (tid == 0 && appended) {
      int* ticket = d_status + kAttnTicketInt;
      __threadfence();
      if (atomicAdd(ticket, 1) == (int)gridDim.x - 1) {
        const int Bt = (int)(gridDim.x / (unsigned)(n_splits * row_tiles * Hkv));
        for (int bb = 0; bb < Bt; ++bb) {
          const int cur = cache_len[bb];
          if (cur >= 0 && cur + T_q <= capacity) cache_len[bb] = cur + T_q;
        }
        *ticket = 0;
      }
    }
  }
  if (warp == kMmaWarp0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

cudaError_t launch_attn_tc4(const samkv_shape_t& s, void* Kc, void* Vc, int capacity, int32_t* cache_len,
                            const void* Q, int T_q, const void* Kq, const void* Vq, float scale, void* O, float* lse,
                            float* part_o, float2* part_ml, const AttnPlan& plan, int* d_status, cudaStream_t stream) {
  const int G = s.n_q_heads / s.n_kv_heads;
  const int rows = T_q * G;
  const int row_tiles = (rows + tc4::kBM - 1) / tc4::kBM;
  const long long blocks = (long long)s.batch * s.n_kv_heads * row_tiles * plan.n_splits;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  CUtensorMap tmK, tmV;
  if (!tc::make_kv_map(&tmK, Kc, capacity, s.batch * s.n_kv_heads) ||
      !tc::make_kv_map(&tmV, Vc, capacity, s.batch * s.n_kv_heads))
    return cudaErrorInvalidValue;
  const bool pair = attn_merges_in_cluster(plan);
  auto kern = pair ? attn_tc4_kernel<true> : attn_tc4_kernel<false>;
  cudaError_t e = pair ? ensure_dynamic_smem<1>(kern, tc4::kSmemBytes) : ensure_dynamic_smem<2>(kern, tc4::kSmemBytes);
  if (e != cudaSuccess) return e;
  // Launched so that it may start while the kernel before it in the stream is still running: barrier set-up and the
  // tensor-memory allocation need nothing from it; one wait precedes every read.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)blocks);
  cfg.blockDim = dim3(tc4::kThreads);
  cfg.dynamicSmemBytes = tc4::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attrs[2];
  attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attrs[0].val.programmaticStreamSerializationAllowed = 1;
  attrs[1].id = cudaLaunchAttributeClusterDimension;
  attrs[1].val.clusterDim.x = 2;
  attrs[1].val.clusterDim.y = 1;
  attrs[1].val.clusterDim.z = 1;
  cfg.attrs = attrs;
  cfg.numAttrs = pair ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, kern, tmK, tmV, cache_len, (const __nv_bfloat16*)Q, (const __nv_bfloat16*)Kq,
                            (const __nv_bfloat16*)Vq, (__nv_bfloat16*)Kc, (__nv_bfloat16*)Vc, (__nv_bfloat16*)O, lse, part_o,
                            part_ml, s.n_q_heads, s.n_kv_heads, T_q, capacity, scale, plan.n_splits, row_tiles, d_status);
}

}  // namespace samkv
