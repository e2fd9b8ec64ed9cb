// pqhsa_select_static: the top-k step for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need a top-k:
// code that runs inside an engine's already-planned memory pool, plugins that are handed
// tensors but no allocator, and latency-critical paths where a driver allocation (which may
// synchronise the whole device) is not acceptable.  pqhsa_select needs a caller-provided
// workspace for its counters and candidate lists; this variant keeps that scratch
// in one fixed array that is part of the library image, so the caller passes only inputs and
// outputs.  The price: a fixed upper size, and one array shared by every call on a device.
#include <mutex>

#include "common.cuh"

namespace pqhsa {

// 16 MiB per GPU, resident from the moment the library is loaded until the process exits.
constexpr size_t kStaticScratchBytes = 16u << 20;
static __device__ __align__(256) unsigned char g_select_scratch[kStaticScratchBytes];

namespace {

constexpr int kMaxDevices = 64;
unsigned char* g_scratch_ptr[kMaxDevices];    // device address of the array, per device
std::mutex g_scratch_mu;

// The array's name is only a host-side handle; kernels need its device address, which
// differs per device.  Looked up once per device, with that device current.
cudaError_t scratch_address(unsigned char** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_scratch_mu);
  if (g_scratch_ptr[dev] == nullptr) {
    unsigned char* p = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_select_scratch);
    if (e != cudaSuccess) return e;
    if (p == nullptr) return cudaErrorInvalidSymbol;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// Only what the top-k kernels touch, packed from offset 0; the first `zero_bytes` bytes are
// the part that must start at zero (status word, counters).
void make_select_layout(const Plan& pl, WsLayout* L) {
  *L = WsLayout{};
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align256(o + bytes); return at; };
  L->zero_begin = 0;
  L->status = take(16);
  L->counters = take((size_t)pl.rows * 16);
  L->zero_bytes = o;
  L->rowstate = take((size_t)pl.rows * 16);
  L->cand = take((size_t)pl.rows * pl.cand_cap * 8);
  L->stage_end = o;
  L->total = o;
}

}  // namespace
}  // namespace pqhsa

using namespace pqhsa;

extern "C" {

size_t pqhsa_select_static_capacity(void) { return kStaticScratchBytes; }

size_t pqhsa_select_static_bytes(const pqhsa_params* params) {
  Plan pl;
  if (make_plan(params, &pl) != PQHSA_OK) return 0;
  WsLayout L;
  make_select_layout(pl, &L);
  return L.total;
}

int pqhsa_select_static(const pqhsa_params* params, const float* scores, const int32_t* seq_lens,
                        int32_t* sel_idx, int32_t* sel_count, float* kth_score, void* stream) {
  Plan pl;
  int rc = make_plan(params, &pl);
  if (rc != PQHSA_OK) return rc;
  if (scores == nullptr || seq_lens == nullptr || sel_idx == nullptr || sel_count == nullptr ||
      kth_score == nullptr || (reinterpret_cast<uintptr_t>(scores) & 15u) != 0)
    return PQHSA_ERR_INVALID_ARG;
  WsLayout L;
  make_select_layout(pl, &L);
  if (L.total > kStaticScratchBytes) return PQHSA_ERR_WORKSPACE;   // shape too large for the array
  unsigned char* scratch = nullptr;
  if (scratch_address(&scratch) != cudaSuccess) return PQHSA_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the array keeps the previous call's contents: clear what the kernels expect to be zero
  if (cudaMemsetAsync(scratch + L.zero_begin, 0, L.zero_bytes, st) != cudaSuccess)
    return PQHSA_ERR_CUDA;
  const cudaError_t e = launch_select(pl, L, reinterpret_cast<char*>(scratch), scores, seq_lens,
                                      sel_idx, sel_count, kth_score, st);
  return e == cudaSuccess ? PQHSA_OK : PQHSA_ERR_CUDA;
}

}  // extern "C"
