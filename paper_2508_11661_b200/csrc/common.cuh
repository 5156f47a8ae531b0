// Shared device/host declarations of the SamKV CUDA library (internal; the public surface is include/samkv.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "samkv.h"

namespace samkv {

// Per-request context tables, passed to kernels by value (no device copy, safe under stream capture).
struct CtxTable {
  int n_ctx;
  int block_size;
  int block_shift;                      // log2(block_size)
  int ctx_off[SAMKV_MAX_CTX + 1];       // token offset of each context on the concatenated axis
  int unit_off[SAMKV_MAX_CTX + 1];      // unit offset of each context
};

// Selection layout: where each context's kept units / kept tokens start.
struct SelTable {
  int sel_off[SAMKV_MAX_CTX + 1];       // prefix sum of k_units
  int slot_off[SAMKV_MAX_CTX + 1];      // prefix sum of kept tokens
  int n_init_units[SAMKV_MAX_CTX];      // protected units at the start of the context
  int first_local_unit[SAMKV_MAX_CTX];  // first unit protected because it overlaps the last n_local tokens
};

struct samkv_ctx_impl {
  int device;
  int sm_count;
  int max_smem_optin;
  char* workspace;
  size_t workspace_bytes;
  int* d_status;  // first word of the workspace
  int attn_share_sm;  // samkv_attn_share_sm(): prefer the prefill attention kernel that leaves room on its SM
};

// ----- launchers implemented in the .cu files (all enqueue on `stream`, return cudaGetLastError) -------
cudaError_t launch_qhat(const samkv_shape_t& s, const void* Q, int T_q, const void* Qloc, int T_loc, int use_bias,
                        float* qhat, cudaStream_t stream);
cudaError_t launch_score(const samkv_shape_t& s, const CtxTable& ct, const void* K, const float* qhat, float* scores,
                         int* d_status, cudaStream_t stream);
cudaError_t launch_select(const samkv_shape_t& s, const CtxTable& ct, const SelTable& st, const float* scores,
                          const int32_t* k_units_host, int max_units, int32_t* sel, int* d_status, cudaStream_t stream);
cudaError_t launch_select_compact(const samkv_shape_t& s, const CtxTable& ct, const SelTable& st, const float* scores,
                                  int max_units, int32_t* sel, const void* K, const void* V, void* Kc, void* Vc,
                                  int capacity, int S, int32_t* cache_len, int32_t* inv_map, cudaStream_t stream);
cudaError_t launch_compact(const samkv_shape_t& s, const CtxTable& ct, const SelTable& st, const void* K, const void* V,
                           const int32_t* sel, void* Kc, void* Vc, int capacity, int S, int32_t* cache_len,
                           int32_t* inv_map, int* d_status, cudaStream_t stream);
cudaError_t launch_update(const samkv_shape_t& s, int L_tot, void* Kc, void* Vc, int capacity, const int32_t* inv_map,
                          const int32_t* tok_ids, int R, const void* Knew, const void* Vnew, int mode, int* d_status,
                          cudaStream_t stream);

cudaError_t launch_topp(const samkv_shape_t& s, const CtxTable& ct, const int* n_init_units, const int* first_local_unit,
                        const float* scores, const int32_t* star_layers, int n_star, const int32_t* max_units,
                        const int32_t* min_units, float* P_out, cudaStream_t stream);
cudaError_t launch_select_cross(const samkv_shape_t& s, const CtxTable& ct, const int* n_init_units,
                                const int* first_local_unit, const float* scores, const int32_t* cand, int K, int S_u,
                                void* scratch, int32_t* sel, int32_t* counts, int max_smem_optin, cudaStream_t stream);
cudaError_t launch_compact_units(const samkv_shape_t& s, const CtxTable& ct, const int* n_init_units,
                                 const int* first_local_unit, const void* K, const void* V, const int32_t* sel, int S_u,
                                 int S, void* Kc, void* Vc, int capacity, int32_t* cache_len, int32_t* inv_map,
                                 int* d_status, cudaStream_t stream);

cudaError_t launch_align(const samkv_shape_t& s, int L_tot, const int32_t* inv_map, const int32_t* tok_ids, int R,
                         uint8_t* flags, int32_t* merged_ids, int32_t* merged_len, int32_t* run_ids, int run_capacity,
                         int32_t* run_len, int* d_status, cudaStream_t stream);

cudaError_t launch_block_means(const samkv_shape_t& s, const CtxTable& ct, const void* K, void* Kbar, int sm_count,
                               cudaStream_t stream);

struct AttnPlan {
  int n_splits;        // KV splits per (batch, kv head, row tile)
  int rows_per_cta;    // packed query rows (T_q * G) per CTA
  size_t partial_bytes;
  int share_sm;        // 128 rows per CTA with the kernel that leaves registers and shared memory to other streams
};
AttnPlan plan_attn(const samkv_shape_t& s, int T_q, int capacity, int sm_count, int share_sm);
// The 128-row tcgen05 kernel with exactly two KV splits merges them inside a two-CTA cluster: no merge kernel.
inline bool attn_merges_in_cluster(const AttnPlan& p) { return p.rows_per_cta == 128 && p.n_splits == 2; }
// Status block of the workspace (256 bytes, zero between calls): int 0 is the device check word, this int counts the
// finished CTAs of an attention grid that bumps cache_len itself.
constexpr int kAttnTicketInt = 32;
cudaError_t launch_attn(const samkv_shape_t& s, int layer, void* Kc, void* Vc, int capacity, int32_t* cache_len,
                        const void* Q, int T_q, const void* Kq, const void* Vq, float scale, void* O, float* lse,
                        void* partial_ws, const AttnPlan& plan, int* d_status, cudaStream_t stream);

// Raises a kernel's dynamic shared-memory limit to `bytes`; the runtime call is made only when this process has not
// yet set at least that much for this kernel on the current device (the setting is per device and sticks), so that
// repeated calls of an entry point cost nothing.  One static slot per instantiation (kTag distinguishes call sites).
// Internal linkage on purpose: with external linkage the slot would be shared between two copies of this library
// loaded into one process (the regular and the debug build), and the second copy would skip its own kernels.
template <int kTag, typename Kernel>
static cudaError_t ensure_dynamic_smem(Kernel kernel, int bytes) {
  constexpr int kMaxDev = 64;
  static int granted[kMaxDev] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < kMaxDev && granted[dev] >= bytes) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && dev >= 0 && dev < kMaxDev) granted[dev] = bytes;
  return e;
}

// ----- small device helpers ---------------------------------------------------------------------------
enum DeviceCheck : int {
  CHECK_OK = 0,
  CHECK_SEL_RANGE = 1,      // a selected unit id lies outside its context, or a recomputed token / its slot is out of range
  CHECK_APPEND_CAPACITY = 2, // cache_len + T_q exceeds the cache capacity
  CHECK_WAIT_TIMEOUT = 3,    // a bounded wait on an mbarrier ran out
  CHECK_SMEM_ALIGNMENT = 4,  // dynamic shared memory not aligned as the tensor-core tiles need
  CHECK_LIST_CAPACITY = 5    // an output list is longer than the capacity the caller gave (it was truncated)
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <typename T>
struct ElemTraits;
template <>
struct ElemTraits<float> {
  static constexpr int kPerVec = 4;  // elements in a 16-byte vector
  __device__ static __forceinline__ void unpack(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  __device__ static __forceinline__ uint4 pack(const float* f) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
  }
};
template <>
struct ElemTraits<__nv_bfloat16> {
  static constexpr int kPerVec = 8;
  __device__ static __forceinline__ void unpack(const uint4& v, float* f) {
    f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
    f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z); f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
  }
  __device__ static __forceinline__ uint32_t pack2(float a, float b) {
    __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&t);
  }
  __device__ static __forceinline__ uint4 pack(const float* f) {
    return make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7]));
  }
};

// Streaming (read-once) 16-byte global load that does not pollute L1.
__device__ __forceinline__ uint4 ld_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream(void* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Programmatic dependent launch: a kernel launched with the programmatic-stream-serialization attribute may start
// once every CTA of the kernel before it in the stream has called pdl_launch_dependents() (or exited); it must call
// pdl_wait() before touching anything that kernel writes.  Both are no-ops in a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Context that owns global index `x` in a prefix table `off[0..n]` (off[c] <= x < off[c+1]).
__device__ __forceinline__ int find_segment(const int* off, int n, int x) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (off[mid] <= x) lo = mid; else hi = mid - 1;
  }
  return lo;
}

}  // namespace samkv
