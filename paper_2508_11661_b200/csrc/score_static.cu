// samkv_score_static: the scoring step for callers that cannot allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a serving engine that has
// handed every byte of HBM to its own pool at start-up, or in a latency-critical section where an
// allocation (which may synchronise the device) is not acceptable.  samkv_score needs scratch for
// the personalised query vectors; here that scratch is a fixed array that lives in the library's
// own device image, so the call needs no handle, no workspace and no allocator.
#include <mutex>

#include "common.cuh"

namespace samkv {
// declared in api.cu: shape validation + context tables without touching the GPU
samkv_status_t build_ctx_table(const samkv_shape_t* shape, CtxTable* ct);
}  // namespace samkv

namespace {

// Scratch for the personalised query vectors q^ [L, Bt, D, Hkv, d] in fp32.  1 MiB per GPU that loads
// the library, held until the process exits.
constexpr size_t kStaticQhatFloats = 256 * 1024;
static __device__ __align__(256) float g_static_qhat[kStaticQhatFloats];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
float* g_qhat_addr[kMaxDevices] = {};   // device address of g_static_qhat, per device, filled on first use

// In host code `g_static_qhat` is only a handle for the runtime, not an address a kernel can use:
// the device address must be asked for, once per device, with that device current.
cudaError_t static_qhat_address(int device, float** out) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_qhat_addr[device] == nullptr) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_qhat);
    if (e != cudaSuccess) return e;
    g_qhat_addr[device] = static_cast<float*>(p);
  }
  *out = g_qhat_addr[device];
  return cudaSuccess;
}

}  // namespace

extern "C" samkv_status_t samkv_score_static(const samkv_shape_t* shape, const void* K, const void* Q, int32_t T_q,
                                             const void* Qloc, int32_t T_loc, int32_t use_bias, float* scores_out,
                                             void* stream) {
  using namespace samkv;
  CtxTable ct;
  samkv_status_t st = build_ctx_table(shape, &ct);
  if (st != SAMKV_OK) return st;
  if (K == nullptr || Q == nullptr || scores_out == nullptr || T_q < 1) return SAMKV_ERR_INVALID_ARG;
  if (Qloc != nullptr && T_loc < 1) return SAMKV_ERR_INVALID_ARG;
  auto misaligned = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
  if (misaligned(K) || misaligned(Q) || misaligned(Qloc) || misaligned(scores_out)) return SAMKV_ERR_INVALID_ARG;
  const size_t need = (size_t)shape->n_layers * shape->batch * shape->n_ctx * shape->n_kv_heads * shape->head_dim;
  if (need > kStaticQhatFloats) return SAMKV_ERR_WORKSPACE;   // beyond SAMKV_STATIC_SCORE_MAX_FLOATS
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return SAMKV_ERR_CUDA;
  float* qhat = nullptr;
  if (static_qhat_address(device, &qhat) != cudaSuccess) return SAMKV_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // qhat_kernel writes every element of the range it uses before score_kernel reads it, so nothing
  // left over from an earlier call can leak into this one and nothing needs clearing.
  if (launch_qhat(*shape, Q, T_q, Qloc, T_loc, use_bias, qhat, s) != cudaSuccess) return SAMKV_ERR_CUDA;
  // no handle, hence no status word: the kernel's bounded waits cannot report here
  return launch_score(*shape, ct, K, qhat, scores_out, nullptr, s) == cudaSuccess ? SAMKV_OK : SAMKV_ERR_CUDA;
}
