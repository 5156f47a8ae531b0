// Cross-layer alignment of the sparse caches (Sec. 3.3): every layer is laid over the union of all layers' kept
// tokens, positions a layer does not keep are blanks, and the two recomputation rules decide per (layer, token)
// whether K/V are recomputed, whether the layer's output is needed, and whether a blank position feeds the
// forward pass from its prefilled entry.  Pure integer work on inv_map and the recompute lists.
#include "common.cuh"

namespace samkv {

constexpr int kAlignThreads = 256;
constexpr uint8_t kFlagKept = 1, kFlagRecompute = 2, kFlagOutput = 4, kFlagPadReuse = 8;

// flags[n, b, t] = "listed for recomputation at layer n" (tentative: the layer must also keep the token).
__global__ void __launch_bounds__(kAlignThreads)
align_mark_kernel(const int32_t* __restrict__ tok_ids, uint8_t* __restrict__ flags, int L, int Bt, int R, int L_tot,
                  int* __restrict__ d_status) {
  const int i = blockIdx.x * kAlignThreads + threadIdx.x;
  if (i >= L * R) return;
  const int n = i / R;
  const int t = tok_ids[i];
  if (t < 0) return;
  if (t >= L_tot) {
    atomicMax(d_status, (int)CHECK_SEL_RANGE);
    return;
  }
  for (int b = 0; b < Bt; ++b) flags[((size_t)n * Bt + b) * L_tot + t] = kFlagRecompute;
}

// One thread per (layer, batch element, token): is the token kept by any head, and is its listing effective.
__global__ void __launch_bounds__(kAlignThreads)
align_kept_kernel(const int32_t* __restrict__ inv_map, uint8_t* __restrict__ flags, int Hkv, int L_tot) {
  const int t = blockIdx.x * kAlignThreads + threadIdx.x;
  const size_t lb = blockIdx.y;                                 // layer * Bt + batch element
  if (t >= L_tot) return;
  const int32_t* row = inv_map + lb * Hkv * L_tot + t;
  bool kept = false;
  for (int h = 0; h < Hkv; ++h) kept = kept || (row[(size_t)h * L_tot] >= 0);
  uint8_t* f = flags + lb * L_tot + t;
  const bool rec = (*f != 0) && kept;
  *f = (kept ? kFlagKept : 0) | (rec ? kFlagRecompute : 0);
}

// One thread per (batch element, token), layers from the top down: rule 1 propagates "recomputed above".
// Layer 0's byte also carries, in kScratchOnAxis, "kept by some layer" for the list kernel; it is cleared afterwards.
constexpr uint8_t kScratchOnAxis = 0x80;
__global__ void __launch_bounds__(kAlignThreads)
align_rules_kernel(uint8_t* __restrict__ flags, int L, int Bt, int L_tot) {
  const int t = blockIdx.x * kAlignThreads + threadIdx.x;
  const int b = blockIdx.y;
  if (t >= L_tot) return;
  bool above = false, on_axis = false;                          // some higher layer recomputes / any layer keeps
#pragma unroll 4
  for (int n = L - 1; n >= 0; --n) {
    uint8_t* f = flags + ((size_t)n * Bt + b) * L_tot + t;
    uint8_t v = *f;
    const bool kept = v & kFlagKept, rec = v & kFlagRecompute;
    if (above) v |= kFlagOutput;
    if (above && !rec && !kept) v |= kFlagPadReuse;
    above = above || rec;
    on_axis = on_axis || kept;
    if (n == 0 && on_axis) v |= kScratchOnAxis;
    *f = v;
  }
}

__global__ void __launch_bounds__(kAlignThreads)
align_clear_kernel(uint8_t* __restrict__ flags, int n) {        // layer 0 occupies the first Bt * L_tot bytes
  const int i = blockIdx.x * kAlignThreads + threadIdx.x;
  if (i < n) flags[i] &= (uint8_t)~kScratchOnAxis;
}

// Ordered lists.  Rows [0, L*Bt): tokens of (layer, batch element) that enter the forward pass (recompute or
// output); rows [L*Bt, L*Bt + Bt): the merged axis of a batch element (kept by any layer).  One CTA per row.
__global__ void __launch_bounds__(kAlignThreads)
align_lists_kernel(const uint8_t* __restrict__ flags, int32_t* __restrict__ run_ids, int32_t* __restrict__ run_len,
                   int32_t* __restrict__ merged_ids, int32_t* __restrict__ merged_len, int L, int Bt, int L_tot,
                   int run_capacity, int* __restrict__ d_status) {
  __shared__ int warp_tot[kAlignThreads / 32];
  const int row = blockIdx.x;
  const bool is_run = row < L * Bt;
  const int b = is_run ? row % Bt : row - L * Bt;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = (L_tot + kAlignThreads - 1) / kAlignThreads;
  const int a = min(tid * per, L_tot), e = min(a + per, L_tot);
  auto member = [&](int t) -> bool {
    if (is_run) return (flags[(size_t)row * L_tot + t] & (kFlagRecompute | kFlagOutput)) != 0;
    return (flags[(size_t)b * L_tot + t] & kScratchOnAxis) != 0;
  };
  int mine = 0;
  for (int t = a; t < e; ++t) mine += member(t);
  int inc = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += v;
  }
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  int before = 0, total = 0;
  for (int i = 0; i < kAlignThreads / 32; ++i) {
    if (i < warp) before += warp_tot[i];
    total += warp_tot[i];
  }
  int pos = before + inc - mine;
  int32_t* out = is_run ? run_ids + (size_t)row * run_capacity : merged_ids + (size_t)b * L_tot;
  const int cap = is_run ? run_capacity : L_tot;
  for (int t = a; t < e; ++t)
    if (member(t)) {
      if (pos < cap) out[pos] = t;
      ++pos;
    }
  for (int i = total + tid; i < cap; i += kAlignThreads) out[i] = -1;          // unused tail of the list
  if (tid == 0) {
    if (is_run) run_len[row] = total; else merged_len[b] = total;
    if (total > cap) atomicMax(d_status, (int)CHECK_LIST_CAPACITY);
  }
}

cudaError_t launch_align(const samkv_shape_t& s, int L_tot, const int32_t* inv_map, const int32_t* tok_ids, int R,
                         uint8_t* flags, int32_t* merged_ids, int32_t* merged_len, int32_t* run_ids, int run_capacity,
                         int32_t* run_len, int* d_status, cudaStream_t stream) {
  const int L = s.n_layers, Bt = s.batch;
  if ((long long)L * Bt > 65535) return cudaErrorInvalidConfiguration;      // (layer, batch) pairs ride on gridDim.y
  cudaError_t e = cudaMemsetAsync(flags, 0, (size_t)L * Bt * L_tot, stream);
  if (e != cudaSuccess) return e;
  if (R > 0)
    align_mark_kernel<<<(L * R + kAlignThreads - 1) / kAlignThreads, kAlignThreads, 0, stream>>>(tok_ids, flags, L, Bt, R,
                                                                                              L_tot, d_status);
  const unsigned tiles = (L_tot + kAlignThreads - 1) / kAlignThreads;
  align_kept_kernel<<<dim3(tiles, L * Bt), kAlignThreads, 0, stream>>>(inv_map, flags, s.n_kv_heads, L_tot);
  align_rules_kernel<<<dim3(tiles, Bt), kAlignThreads, 0, stream>>>(flags, L, Bt, L_tot);
  align_lists_kernel<<<L * Bt + Bt, kAlignThreads, 0, stream>>>(flags, run_ids, run_len, merged_ids, merged_len, L, Bt,
                                                               L_tot, run_capacity, d_status);
  align_clear_kernel<<<(Bt * L_tot + kAlignThreads - 1) / kAlignThreads, kAlignThreads, 0, stream>>>(flags, Bt * L_tot);
  return cudaGetLastError();
}

}  // namespace samkv
