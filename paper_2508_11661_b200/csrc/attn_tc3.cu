// Warp-specialised tcgen05 attention over the compact cache for prefill chunks (Sec. 3.3), d = 128, with the
// score tile double-buffered in tensor memory: the variant that leaves room on its SM.
//
// This kernel is slower on its own than the one with two tile groups (attn_tc4.cu), but it runs 320 threads with
// 128 registers and 200 KB of shared memory, so about eight small copy CTAs (the gather and update kernels of the
// next layers) fit beside each of its CTAs.  A caller that runs such kernels on another stream while attention is
// in flight asks for it with samkv_attn_share_sm(); everyone else gets the faster kernel.
//
// One CTA per SM: one 128-row query tile (packed rows of one (batch, kv head); row r = token r / G, group member
// r % G) and one KV split, walked in tiles of 128 slots.  Roles:
//   warps 0-7   softmax: two threads per row (warp w and warp w + 4 share the tensor-memory lanes of rows
//               32 (w % 4) .., thread halves own score columns [0,64) and [64,128)); each reads its half of the S
//               row twice (maximum, then exponentials), the halves exchange their maxima through shared memory,
//               and P goes back as packed bf16 over S columns the same thread has already consumed
//               (slots [0,64) -> columns [0,32), slots [64,128) -> columns [64,96) of the S buffer); O is rescaled
//               in tensor memory only when a row's reference maximum grew by more than 2^8
//   warp  8     one thread issues every tcgen05.mma.  S(j+2) = Q K(j+2)^T is issued right behind O += P(j) V(j)
//               into the S buffer that P(j) occupied, so while the softmax warps work on S(j+1) the tensor pipe
//               already produces the tile after it: the softmax never waits for the round trip
//               P ready -> O += P V -> next S.
//   warp  9     loader: K (3 stages) and V (2 stages) tiles arrive by TMA (cp.async.bulk.tensor, 128-byte swizzle)
// Tensor memory: S buffers [0,128) and [128,256), O [256,384).
// With exactly two KV splits the grid is launched in clusters of two CTAs (the two splits of one query tile): the
// CTAs swap the (m, l, O) of half of the rows each through distributed shared memory between two cluster barriers and
// each writes the final result of its half; every thread of both CTAs walks through both barriers on every path.
// All hand-offs are mbarriers polled by one lane per warp; every wait is bounded and a timeout is recorded as a
// device check, after which the CTA drains and frees its tensor memory.  The TMA loads read this GPU's memory only
// and use no multicast.
#include "tc_common.cuh"

namespace samkv {
namespace tc3 {
using namespace tc;

constexpr int kBM = 128, kBN = 128, kD = 128;
constexpr int kStagesK = 3, kStagesV = 2;
constexpr int kParts = 2;                     // threads per row: each owns kPartCols score columns and O columns
constexpr int kPartCols = kBN / kParts;
constexpr int kSoftmaxWarps = 4 * kParts;
constexpr int kMmaWarp = kSoftmaxWarps, kLoadWarp = kSoftmaxWarps + 1;
constexpr int kThreads = (kSoftmaxWarps + 2) * 32;
constexpr int kQBytes = kBM * kD * 2;         // 32 KB
constexpr int kTileBytes = kBN * kD * 2;      // 32 KB per K or V tile
constexpr int kOffQ = 0;
constexpr int kOffK = kQBytes;
constexpr int kOffV = kOffK + kStagesK * kTileBytes;
constexpr int kOffX = kOffV + kStagesV * kTileBytes;   // exchange: row maxima [2 parities][parts][128], row sums [parts][128]
constexpr int kOffBar = kOffX + (2 * kParts * kBM + kParts * kBM) * 4;
constexpr int kSmemBytes = kOffBar + 256;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemO = 256;

enum Bar {
  K_FULL = 0, K_EMPTY = 3, V_FULL = 6, V_EMPTY = 8, KV_TMA = 10, S_FULL = 11, P_READY = 13, PV_DONE = 15, O_FINAL = 16,
  Q_READY = 17, N_BARS = 18
};

}  // namespace tc3

// kPair: the grid is launched in clusters of two CTAs, the two KV splits of one (batch, kv head, query tile).  The
// CTA of the second split hands its (m, l, O) to the first one through distributed shared memory, which writes the
// final rows: no partial results in global memory and no merge kernel.  The cache length of an appended chunk is then
// bumped by the last CTA of the grid to finish (a counter in the workspace's status block).
template <bool kPair>
__global__ void __launch_bounds__(tc3::kThreads, 1)
attn_tc3_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                int32_t* cache_len, const __nv_bfloat16* __restrict__ Q,
                __nv_bfloat16* __restrict__ O, float* __restrict__ lse, float* __restrict__ part_o,
                float2* __restrict__ part_ml, int Hq, int Hkv, int T_q, int capacity, int appended, float scale,
                int n_splits, int row_tiles, int* __restrict__ d_status) {
  using namespace tc3;
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
  float* x_max = reinterpret_cast<float*>(smem_raw + kOffX);          // [parity][half][row]
  float* x_sum = x_max + 2 * kParts * kBM;                            // [part][row]
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

  // ---- set-up ----
  if (tid == 0) {
    for (int i = 0; i < kStagesK; ++i) { mbar_init(bar(K_FULL + i), 1); mbar_init(bar(K_EMPTY + i), 1); }
    for (int i = 0; i < kStagesV; ++i) { mbar_init(bar(V_FULL + i), 1); mbar_init(bar(V_EMPTY + i), 1); }
    mbar_init(bar(KV_TMA), 1);
    mbar_init(bar(PV_DONE), 1);
    mbar_init(bar(O_FINAL), 1);
    mbar_init(bar(Q_READY), kSoftmaxWarps);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(S_FULL + i), 1);
      mbar_init(bar(P_READY + i), kSoftmaxWarps);
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

  if (warp < kSoftmaxWarps) {
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    fence_proxy_async();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar(Q_READY));
  }

  if (warp == kLoadWarp) {
    // ================= loader: K(0), K(1), then V(j), K(j+2) in the order the MMA thread asks for them =================
    auto load_k = [&](int j) {
      const int s = j % kStagesK;
      const uint32_t round = (uint32_t)(j / kStagesK);
      const int j0 = (tile0 + j) * kBN;
      mbar_wait_warp(bar(K_EMPTY + s), (round & 1) ^ 1, s_fail);
      if (lane == 0) {
        mbar_expect_tx(bar(K_FULL + s), kTileBytes);
        tma_load_3d(sK + s * kTileBytes, &tmK, 0, j0, bh, bar(K_FULL + s));
        tma_load_3d(sK + s * kTileBytes + kBN * 128, &tmK, 64, j0, bh, bar(K_FULL + s));
      }
      __syncwarp();
    };
    auto load_v = [&](int j) {
      const int s = j % kStagesV;
      const uint32_t round = (uint32_t)(j / kStagesV);
      const int j0 = (tile0 + j) * kBN;
      mbar_wait_warp(bar(V_EMPTY + s), (round & 1) ^ 1, s_fail);
      const bool partial = j0 + kBN > total;                     // V rows past `total` must read as zero
      const uint32_t target = partial ? bar(KV_TMA) : bar(V_FULL + s);
      if (lane == 0) {
        mbar_expect_tx(target, kTileBytes);
        tma_load_3d(sV + s * kTileBytes, &tmV, 0, j0, bh, target);
        tma_load_3d(sV + s * kTileBytes + kBN * 128, &tmV, 64, j0, bh, target);
      }
      if (partial) {                                              // at most once per CTA: the last tile of the cache
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
    };
    if (nt > 0) load_k(0);
    if (nt > 1) load_k(1);
    for (int j = 0; j < nt; ++j) {
      load_v(j);
      if (j + 2 < nt) load_k(j + 2);
    }
    if constexpr (kPair) { pair_sync(); pair_sync(); }
  } else if (warp == kMmaWarp) {
    // ================= MMA issuer =================
    if (lane == 0 && nt > 0) {
      constexpr uint32_t kIdescS = instr_desc(kBM, kBN, false);
      constexpr uint32_t kIdescO = instr_desc(kBM, kD, true);
      // Descriptors are built once; per instruction only the 14-bit start-address field (16-byte units) moves.
      const uint64_t dQ = smem_desc(sQ, 16, 1024), dK = smem_desc(sK, 16, 1024);
      const uint64_t dV = smem_desc(sV, kBN * 128, 1024);
      auto issue_s = [&](int j) {                               // S(j) = Q K(j)^T into buffer j & 1: 8 k-steps over d
        const int s = j % kStagesK;
        mbar_wait(bar(K_FULL + s), (uint32_t)((j / kStagesK) & 1), s_fail);
        tc_fence_after();
        const uint64_t b0 = dK + (uint64_t)(s * (kTileBytes >> 4));
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
          const uint32_t aoff = ((ks >> 2) * (kBM * 128) + (ks & 3) * 32) >> 4;
          const uint32_t boff = ((ks >> 2) * (kBN * 128) + (ks & 3) * 32) >> 4;
          mma_ss(tmem + (j & 1) * kBN, dQ + aoff, b0 + boff, kIdescS, ks > 0);
        }
        mma_commit(bar(S_FULL + (j & 1)));
        mma_commit(bar(K_EMPTY + s));
      };
      auto issue_pv = [&](int j) {                              // O += P(j) V(j): 8 k-steps over the 128 slots
        const int s = j % kStagesV;
        mbar_wait(bar(V_FULL + s), (uint32_t)((j / kStagesV) & 1), s_fail);
        mbar_wait(bar(P_READY + (j & 1)), (uint32_t)((j >> 1) & 1), s_fail);
        tc_fence_after();
        const uint64_t b0 = dV + (uint64_t)(s * (kTileBytes >> 4));
        const uint32_t pbase = tmem + (j & 1) * kBN;
#pragma unroll
        for (int ks = 0; ks < kBN / 16; ++ks) {
          constexpr int kStepsPerPart = 8 / kParts;                         // 16-slot steps inside one thread's columns
          const uint32_t pcol = (ks / kStepsPerPart) * kPartCols + (ks % kStepsPerPart) * 8;   // where the softmax threads put P
          mma_ts(tmem + kTmemO, pbase + pcol, b0 + ((ks * 16 * 128) >> 4), kIdescO, (j > 0) | (ks > 0));
        }
        mma_commit(bar(PV_DONE));
        mma_commit(bar(V_EMPTY + s));
      };
      mbar_wait(bar(Q_READY), 0, s_fail);
      issue_s(0);
      if (nt > 1) issue_s(1);
      for (int j = 0; j < nt; ++j) {
        issue_pv(j);
        if (j + 2 < nt) issue_s(j + 2);       // overwrites the buffer P(j) sat in; the tensor pipe keeps issue order
      }
      mma_commit(bar(O_FINAL));
    }
    __syncwarp();
    if constexpr (kPair) { pair_sync(); pair_sync(); }
  } else {
    // ================= softmax warps =================
    const int wl = warp & 3;                                    // tensor-memory lane quarter
    const int part = warp >> 2;                                 // score / output columns [kPartCols part, +kPartCols)
    const int row_in_tile = wl * 32 + lane;
    const int my_row = row_base + row_in_tile;
    const uint32_t lane_addr = tmem + ((uint32_t)(wl * 32) << 16);
    const uint32_t tO = lane_addr + kTmemO + part * kPartCols;  // this thread's part of the O row
    const int vis = len + (n_app ? min(my_row, rows_total - 1) / G + 1 : 0);
    const float sl2 = scale * kLog2e;
    float m = -INFINITY, l = 0.f;
    auto row_barrier = [&]() {                                  // the kParts warps that share these 32 rows
      asm volatile("bar.sync %0, %1;" ::"r"(1 + wl), "n"(kParts * 32) : "memory");
    };

    for (int j = 0; j < nt; ++j) {
      const int buf = j & 1;
      const uint32_t tS = lane_addr + buf * kBN + part * kPartCols;   // this thread's score columns
      mbar_wait_warp(bar(S_FULL + buf), (uint32_t)((j >> 1) & 1), s_fail);
      tc_fence_after();
      const int j0 = (tile0 + j) * kBN + part * kPartCols;      // slot of this thread's first column
      const bool masked = j0 + kPartCols > vis;
      // pass 1: maximum of this part of the row, then the other parts' through shared memory
      float sv[kPartCols];
#pragma unroll
      for (int c0 = 0; c0 < kPartCols; c0 += 32) tmem_ld32_nowait(tS + c0, sv + c0);
      tmem_wait_ld();
      if (masked) {
#pragma unroll
        for (int i = 0; i < kPartCols; ++i)
          if (j0 + i >= vis) sv[i] = -INFINITY;
      }
      float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
      for (int i = 0; i < kPartCols; i += 4) {
        mx0 = fmaxf(mx0, sv[i]); mx1 = fmaxf(mx1, sv[i + 1]); mx2 = fmaxf(mx2, sv[i + 2]); mx3 = fmaxf(mx3, sv[i + 3]);
      }
      float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
      x_max[(buf * kParts + part) * kBM + row_in_tile] = mx;
      row_barrier();
#pragma unroll
      for (int pp = 0; pp < kParts; ++pp) mx = fmaxf(mx, x_max[(buf * kParts + pp) * kBM + row_in_tile]);
      const float m_cand = fmaxf(m, mx * sl2);
      const bool grow = (m_cand - m > kRescaleThreshold) || (m == -INFINITY && m_cand > -INFINITY);
      const float m_use = grow ? m_cand : m;
      const float mu = (m_use == -INFINITY) ? 0.f : m_use;
      const float corr = grow ? fast_exp2(m - mu) : 1.0f;
      // rescale this part of O when some row of this warp moved its reference maximum; O must be at rest:
      // O += P(j-1) V(j-1) complete, and O += P(j) V(j) cannot start before this warp's P_READY arrival below
      if (j > 0 && __any_sync(0xffffffffu, grow)) {
        mbar_wait_warp(bar(PV_DONE), (uint32_t)((j - 1) & 1), s_fail);
        tc_fence_after();
#pragma unroll 1
        for (int c0 = 0; c0 < kPartCols; c0 += 32) {
          float o[32];
          tmem_ld32(tO + c0, o);
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] *= corr;
          tmem_st32(tO + c0, o);
        }
      }
      // pass 2: P = exp2(S * scale - m), rounded to bf16, written over S columns this thread has consumed
      // (32 probabilities -> 16 columns; the thread's probabilities land in the first half of its columns)
      float ps0 = 0.f, ps1 = 0.f, ps2 = 0.f, ps3 = 0.f;
#pragma unroll
      for (int c0 = 0; c0 < kPartCols; c0 += 32) {
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
          const float p0 = fast_exp2(fmaf(sv[c0 + i], sl2, -mu));
          const float p1 = fast_exp2(fmaf(sv[c0 + i + 1], sl2, -mu));
          const float p2 = fast_exp2(fmaf(sv[c0 + i + 2], sl2, -mu));
          const float p3 = fast_exp2(fmaf(sv[c0 + i + 3], sl2, -mu));
          // the denominator sums the rounded values, i.e. exactly what the tensor core multiplies with V (here the
          // conversion instruction plus two integer operations per pair is cheaper than rounding on the integer pipe)
          const uint32_t k01 = pack_bf16(p0, p1), k23 = pack_bf16(p2, p3);
          pk[i >> 1] = k01;
          pk[(i >> 1) + 1] = k23;
          ps0 += __uint_as_float(k01 << 16); ps1 += __uint_as_float(k01 & 0xffff0000u);
          ps2 += __uint_as_float(k23 << 16); ps3 += __uint_as_float(k23 & 0xffff0000u);
        }
        tmem_st16(tS + (c0 >> 1), pk);
      }
      l = l * corr + ((ps0 + ps1) + (ps2 + ps3));
      m = m_use;
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(P_READY + buf));
    }
    if (nt > 0) {
      mbar_wait_warp(bar(O_FINAL), 0, s_fail);
      tc_fence_after();
    }
    // ---- the row's denominator: the parts add up in part order (same m in all of them by construction) ----
    x_sum[part * kBM + row_in_tile] = l;
    row_barrier();
    float l_row = 0.f;
#pragma unroll
    for (int pp = 0; pp < kParts; ++pp) l_row += x_sum[pp * kBM + row_in_tile];
    if constexpr (kPair) {
      // ---- merge of the two KV splits inside the cluster ----
      // Exchange area in the first CTA's K ring: O parts [part][row][kPartCols] fp32 with the 16-byte chunks of a row
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
          if (nt > 0) {
            tmem_ld32(tO + c0, o);
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = 0.f;
          }
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
          if (nt > 0) {
            tmem_ld32(tO + c0, o);
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = 0.f;
          }
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
      if (nt > 0) {
        tmem_ld32(tO + c0, o);
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = 0.f;
      }
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
  if (warp == kMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

cudaError_t launch_attn_tc3(const samkv_shape_t& s, const void* Kc, const void* Vc, int capacity, int32_t* cache_len,
                            const void* Q, int T_q, int appended, float scale, void* O, float* lse, float* part_o,
                            float2* part_ml, const AttnPlan& plan, int* d_status, cudaStream_t stream) {
  const int G = s.n_q_heads / s.n_kv_heads;
  const int rows = T_q * G;
  const int row_tiles = (rows + tc3::kBM - 1) / tc3::kBM;
  const long long blocks = (long long)s.batch * s.n_kv_heads * row_tiles * plan.n_splits;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  CUtensorMap tmK, tmV;
  if (!tc::make_kv_map(&tmK, Kc, capacity, s.batch * s.n_kv_heads) ||
      !tc::make_kv_map(&tmV, Vc, capacity, s.batch * s.n_kv_heads))
    return cudaErrorInvalidValue;
  const bool pair = attn_merges_in_cluster(plan);
  auto kern = pair ? attn_tc3_kernel<true> : attn_tc3_kernel<false>;
  cudaError_t e = pair ? ensure_dynamic_smem<3>(kern, tc3::kSmemBytes) : ensure_dynamic_smem<4>(kern, tc3::kSmemBytes);
  if (e != cudaSuccess) return e;
  // Launched so that it may start while the kernel before it in the stream (the append of the chunk) is still
  // running: set-up and the Q loads need nothing from it; one wait precedes everything that does.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)blocks);
  cfg.blockDim = dim3(tc3::kThreads);
  cfg.dynamicSmemBytes = tc3::kSmemBytes;
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
  return cudaLaunchKernelEx(&cfg, kern, tmK, tmV, cache_len, (const __nv_bfloat16*)Q, (__nv_bfloat16*)O, lse, part_o,
                            part_ml, s.n_q_heads, s.n_kv_heads, T_q, capacity, appended, scale, plan.n_splits, row_tiles,
                            d_status);
}

}  // namespace samkv
