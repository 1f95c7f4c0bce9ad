// sp_gemm_noalloc: the swizzled GEMM for callers that must not allocate device memory.
//
// sp_gemm keeps two pieces of scratch in memory it obtains with cudaMalloc: the tile
// table that non-arithmetic orders (space-filling curves on irregular grids, caller
// tables) are served from, and the status word bounded device waits report into.  Some
// callers cannot tolerate that: a serving process that has handed the whole device to
// its own memory pool (a library cudaMalloc then fails, or eats into a budget somebody
// else accounted for), or a latency-critical loop in which an allocation's implicit
// device-wide synchronisation is not acceptable.  For them the same kernel runs here
// with both pieces of scratch in a fixed array that is part of the library image.
//
// The array below lives in every CUDA context that loads the library, from load until
// the process exits (about 257 KiB per device).  Its name is a host-side handle, not a
// device address: the address is looked up once per device with cudaGetSymbolAddress
// and that pointer is what the kernels receive.
#include <string.h>

#include <mutex>
#include <vector>

#include "internal.h"

namespace sp {

constexpr int kNoAllocMaxTiles = 65536;                   // largest tile count this entry point accepts
constexpr int kNoAllocHeaderWords = 64;                   // word 0: status; rest unused (keeps the table 256-byte aligned)
constexpr int kNoAllocWords = kNoAllocHeaderWords + kNoAllocMaxTiles;

static __device__ __align__(256) int32_t g_noalloc_scratch[kNoAllocWords];

// Device code may name the array directly; this is how the status word is cleared.
__global__ void noalloc_clear_status() { g_noalloc_scratch[0] = 0; }

constexpr int kMaxDevices = 64;
static std::mutex g_noalloc_mu;
static int32_t* g_noalloc_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device; looked up on first use.
static int noalloc_scratch(int dev, int32_t** out) {
  if (dev < 0 || dev >= kMaxDevices) { set_error("device index %d out of range", dev); return SP_ERR_DEVICE; }
  std::lock_guard<std::mutex> lock(g_noalloc_mu);
  if (!g_noalloc_ptr[dev]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess || !p) {
      set_error("cudaGetSymbolAddress(scratch) failed: %s", cudaGetErrorString(e));
      return SP_ERR_CUDA;
    }
    g_noalloc_ptr[dev] = static_cast<int32_t*>(p);
  }
  *out = g_noalloc_ptr[dev];
  return SP_OK;
}

}  // namespace sp

using namespace sp;

extern "C" int sp_gemm_noalloc(const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t K, int scheme,
                               const sp_params* params, void* stream, int32_t* status_host) {
  int tile_m, tile_n, out_f32, b_nk;
  int rc = validate_gemm_args(A, B, C, M, N, K, params, &tile_m, &tile_n, &out_f32, &b_nk);
  if (rc != SP_OK) return rc;

  if (params && (params->flags & SP_FLAG_STREAM_K)) {
    set_error("SP_FLAG_STREAM_K needs a workspace and is not available in sp_gemm_noalloc");
    return SP_ERR_INVALID_ARG;
  }
  if (params && (params->flags & SP_FLAG_CLC)) {
    set_error("SP_FLAG_CLC is not available in sp_gemm_noalloc");
    return SP_ERR_INVALID_ARG;
  }
  if (params && (params->flags & SP_FLAG_OVERLAP)) {
    set_error("SP_FLAG_OVERLAP is not available in sp_gemm_noalloc (its scratch is rewritten by every call)");
    return SP_ERR_INVALID_ARG;
  }
  GemmCall call;
  memset(&call, 0, sizeof call);
  rc = resolve_sched(M, N, tile_m, tile_n, scheme, params, &call.sched);
  if (rc != SP_OK) return rc;
  if (call.sched.T > kNoAllocMaxTiles) {
    set_error("sp_gemm_noalloc handles at most %d tiles; this problem has %d (use a larger tile or sp_gemm)",
              kNoAllocMaxTiles, call.sched.T);
    return SP_ERR_UNSUPPORTED;
  }
  std::vector<int32_t> host_perm;   // host memory only; the bijectivity gate of every entry point
  rc = build_perm_host(call.sched, params ? params->custom_perm : nullptr, host_perm);
  if (rc != SP_OK) return rc;

  int ndev = 0, dev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) { cudaGetLastError(); set_error("no CUDA device"); return SP_ERR_DEVICE; }
  if (cudaGetDevice(&dev) != cudaSuccess) { set_error("cudaGetDevice failed"); return SP_ERR_CUDA; }
  if (cudaSetDevice(dev) != cudaSuccess) { set_error("cudaSetDevice failed"); return SP_ERR_CUDA; }   // binds the context to this thread (no allocation)
  int32_t* scratch = nullptr;
  rc = noalloc_scratch(dev, &scratch);
  if (rc != SP_OK) return rc;
  int32_t* status_dev = scratch;                        // word 0
  int32_t* table_dev = scratch + kNoAllocHeaderWords;   // T entries, rewritten by every call that needs a table
  cudaStream_t st = (cudaStream_t)stream;

  // The array keeps whatever the previous call left: the status word must start at zero.
  noalloc_clear_status<<<1, 1, 0, st>>>();
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_error("clearing the status word failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
  call.perm_dev = nullptr;
  if (call.sched.use_table) {
    if (scheme == kCustom) {
      e = cudaMemcpyAsync(table_dev, host_perm.data(), sizeof(int32_t) * (size_t)call.sched.T, cudaMemcpyHostToDevice, st);
      if (e == cudaSuccess) e = cudaStreamSynchronize(st);   // host_perm is pageable and dies with this call
    } else {
      e = launch_build_perm(call.sched, table_dev, st);
    }
    if (e != cudaSuccess) { set_error("filling the tile table failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
    call.perm_dev = table_dev;
  }
  call.A = A; call.B = B; call.C = C; call.M = M; call.N = N; call.K = K;
  call.tile_m = tile_m; call.tile_n = tile_n; call.out_f32 = out_f32; call.b_nk = b_nk;
  call.status_dev = status_dev;
  call.trace_dev = nullptr;
  call.stream = st;
  rc = launch_gemm(call);
  if (rc != SP_OK) return rc;
  if (status_host) {
    int32_t word = 0;
    e = cudaMemcpyAsync(&word, status_dev, sizeof word, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) { set_error("reading the status word failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
    *status_host = word;
    if (word != 0) { set_error("a device-side wait expired (status word 0x%x)", word); return SP_ERR_TIMEOUT; }
  }
  return SP_OK;
}
