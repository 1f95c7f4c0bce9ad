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

// What the table part of the array holds on each device: a call that needs the same table again (the same order on the
// same grid, or the same caller table) neither rebuilds nor re-uploads it.  Valid under this entry point's contract
// that calls on one device do not overlap.
struct NoAllocTable { bool valid; Sched key; uint64_t custom_hash; };
static NoAllocTable g_noalloc_table[kMaxDevices] = {};

static uint64_t table_hash(const int32_t* v, int n) {
  uint64_t h = 1469598103934665603ull;
  for (int i = 0; i < n; ++i) { h ^= (uint32_t)v[i]; h *= 1099511628211ull; }
  return h;
}

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

  if (params && (params->flags & (SP_FLAG_STREAM_K | SP_FLAG_CLC | SP_FLAG_OVERLAP | SP_FLAG_DIE_PINNED))) {
    // STREAM_K needs a workspace and DIE_PINNED its counters (both allocated by sp_gemm); OVERLAP and CLC launches may
    // run beside the call before them, which would rewrite the shared array under a running kernel
    set_error("sp_gemm_noalloc accepts SP_FLAG_SERPENTINE, SP_FLAG_K_ALTERNATE and SP_FLAG_HINT_* only (got 0x%x)", params->flags);
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
  // The bijectivity gate of every entry point, in host memory only.  An order that passed once on this grid is
  // remembered; a caller table is checked on every call (its contents may have changed).
  std::vector<int32_t> host_perm;
  if (scheme == kCustom || !already_validated(call.sched)) {
    rc = build_perm_host(call.sched, params ? params->custom_perm : nullptr, host_perm);
    if (rc != SP_OK) return rc;
    if (scheme != kCustom) remember_validated(call.sched);
  }

  int dev = 0;
  rc = current_device(&dev);   // device present, sm_100, context bound to this thread: no allocation
  if (rc != SP_OK) return rc;
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
    const uint64_t h = scheme == kCustom ? table_hash(host_perm.data(), call.sched.T) : 0;
    bool have;
    {
      std::lock_guard<std::mutex> lock(g_noalloc_mu);
      const NoAllocTable& t = g_noalloc_table[dev];
      have = t.valid && memcmp(&t.key, &call.sched, sizeof(Sched)) == 0 && t.custom_hash == h;
      g_noalloc_table[dev].valid = false;   // until the new contents are queued
    }
    if (!have) {
      if (scheme == kCustom) {
        e = cudaMemcpyAsync(table_dev, host_perm.data(), sizeof(int32_t) * (size_t)call.sched.T, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);   // host_perm is pageable and dies with this call
      } else {
        e = launch_build_perm(call.sched, table_dev, st);
      }
      if (e != cudaSuccess) { set_error("filling the tile table failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
    }
    {
      std::lock_guard<std::mutex> lock(g_noalloc_mu);
      g_noalloc_table[dev].key = call.sched; g_noalloc_table[dev].custom_hash = h; g_noalloc_table[dev].valid = true;
    }
    call.perm_dev = table_dev;
  }
  call.A = A; call.B = B; call.C = C; call.M = M; call.N = N; call.K = K;
  call.tile_m = tile_m; call.tile_n = tile_n; call.out_f32 = out_f32; call.b_nk = b_nk;
  call.status_dev = status_dev;
  call.trace_dev = nullptr;
  rc = apply_memory_flags(params, &call);
  if (rc != SP_OK) return rc;
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
