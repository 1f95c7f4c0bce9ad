// Internal declarations shared by the translation units of libswizzleperf.so.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/swizzleperf.h"
#include "remap.cuh"

namespace sp {

// Largest tile count any entry point accepts, and largest grid side for curve orders
// (their enclosing square has 4^k cells, all of which are visited once).
constexpr int64_t kMaxTiles = 1 << 24;
constexpr int kMaxCurveSide = 4096;

// Stream-K workspace of one stream: a flag per (unit, CTA, lane quarter) and one fp32 partial tile per unit.
// 148 CTAs x 128 rows x 256 columns covers every tile shape up to 256x256 on every unit count.
constexpr size_t kSkFlagBytes = 4096;
constexpr size_t kSkWorkspaceBytes = (size_t)148 * 128 * 256 * 4;

void set_error(const char* fmt, ...);

// Per-function set-up that CUDA keeps per device (cudaFuncSetAttribute): true the first time it is asked for the
// current device with this mask.  A lost race only repeats a harmless call.
inline bool first_use_on_this_device(uint64_t& done_mask) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return true;
  const uint64_t bit = 1ull << (dev & 63);
  if (done_mask & bit) return false;
  done_mask |= bit;
  return true;
}

// The current device, after checking (once per host thread and device) that it exists, is sm_100 and has its primary
// context bound to this thread.  Returns an sp_status.  Allocates nothing.
int current_device(int* dev);

// Validates sizes and parameters and fills `out`.  Returns an sp_status.
int resolve_sched(int64_t M, int64_t N, int32_t tileM, int32_t tileN, int scheme, const sp_params* params, Sched* out);

// Argument checks shared by every GEMM entry point (NULL, sizes, struct version, tile shape, dtype/layout flags,
// alignment); fills the resolved tile shape and flags.  Returns an sp_status.
int validate_gemm_args(const void* A, const void* B, const void* C, int64_t M, int64_t N, int64_t K, const sp_params* params,
                       int* tile_m, int* tile_n, int* out_f32, int* b_nk);

// Evaluates the remap on the host (closed forms, curve walks, caller table) and checks
// that it is a bijection.  Returns SP_OK or SP_ERR_NOT_BIJECTIVE / SP_ERR_INVALID_ARG.
int build_perm_host(const Sched& sched, const int32_t* custom, std::vector<int32_t>& perm);

// Orders (grid, scheme, parameters) that have passed the bijectivity gate, so that repeated calls do no O(T) host work.
bool already_validated(const Sched& c);
void remember_validated(const Sched& c);

// Device evaluation of the same remap into out_dev (T entries).  Not valid for kCustom.
cudaError_t launch_build_perm(const Sched& sched, int32_t* out_dev, cudaStream_t stream);

struct GemmCall {
  const void* A;
  const void* B;
  void* C;
  int64_t M, N, K;
  int tile_m, tile_n;
  int out_f32;
  int b_nk;
  Sched sched;
  const int32_t* perm_dev;  // table for non-arithmetic schemes, else nullptr
  int32_t* status_dev;      // device status word
  int32_t* die_count_dev;   // die-pinned launches: a set of five device counters nobody else uses while this launch runs
  int pinned;               // die-pinned scheduling (SP_DIE_SPLIT + SP_FLAG_DIE_PINNED)
  int steal;                // SP_FLAG_STEAL: per-half ticket queues, an idle half takes the other's tickets (with pinned)
  int half0;                // slots in half 0
  int sms_on_die[2];
  uint32_t die_mask[8];
  sp_trace_rec* trace_dev;  // nullptr unless tracing
  int stream_k;             // SP_FLAG_STREAM_K: split the tail wave along k
  int clc;                  // SP_FLAG_CLC: one cluster per tile, tiles of unstarted clusters taken over by running ones
  int hint_a, hint_b, hint_c;   // SP_FLAG_HINT_*: L2 eviction priority of A loads, B loads, C stores (0 none, 1 first, 2 last)
  int k_alternate;          // SP_FLAG_K_ALTERNATE: odd pieces of work of a unit walk k downwards
  int overlap;              // SP_FLAG_OVERLAP: launch with programmatic stream serialisation, never wait for the predecessor
  int32_t* sk_flags_dev;    // kSkFlagBytes of flags, zero when allocated
  int32_t sk_epoch;         // value the flags take in this launch: 1, 2, ... per workspace
  float* sk_ws_dev;         // kSkWorkspaceBytes of partial tiles
  cudaStream_t stream;
};

// Fills the fields of `call` that SP_FLAG_K_ALTERNATE and SP_FLAG_HINT_* set.  Returns an sp_status.
int apply_memory_flags(const sp_params* params, GemmCall* call);

// Number of persistent units (CTAs or CTA pairs) for this tile shape on the current device.
int gemm_units(int tile_m, int tile_n, int64_t T);
// Encodes tensor maps and launches the kernel.  Returns an sp_status.
int launch_gemm(const GemmCall& call);

// Tensor map of a row-major [rows, cols] matrix of 2-byte (or, with f32, 4-byte) elements with boxes of
// box_rows x 128 bytes and the 128-byte shared-memory swizzle.  `m` is a CUtensorMap.
int make_map(struct CUtensorMap_st* m, const void* base, int64_t rows, int64_t cols, int box_rows, bool f32);
int make_map_plain(struct CUtensorMap_st* m, const void* base, int64_t rows, int64_t cols, int box_rows, int box_cols);
int launch_stencil(const void* in, void* out, int64_t M, int64_t N, float c_center, float c_neighbor, const Sched& sched,
                   const int32_t* perm_dev, int32_t* status_dev, cudaStream_t stream);
int launch_transpose(const void* in, void* out, int64_t M, int64_t N, const Sched& sched, const int32_t* perm_dev,
                     int32_t* status_dev, cudaStream_t stream);
int softmax_rows_per_block(int64_t N);   // single pass: rows of one block, 0 when a row does not fit a buffer
int launch_softmax(const void* in, void* out, int64_t M, int64_t N, int mode, const Sched& sched, const int32_t* perm_dev,
                   float* partial_dev, int32_t* status_dev, cudaStream_t stream);
int selftest_timeout(int32_t* status_dev, int timeout_us, int32_t* code_host, int64_t* waited_us_host);
int probe_dispatch(int n_blocks, int cluster, int32_t* smid_host, uint64_t* start_host);
int probe_topology(int32_t* sm_to_die_host, int32_t* n_sm, float* confidence, uint32_t* lat_host);
int probe_l2_capacity(int n_sizes, const int64_t* sizes_bytes, int half, const uint32_t* die_mask_host, float* gbps_out);
// Size of half 0 of a DIE_SPLIT schedule, in slots.
inline int die_split_half0(const Sched& c) {
  return c.axis == 0 ? ((c.Tm + 1) / 2) * c.Tn : ((c.Tn + 1) / 2) * c.Tm;
}

}  // namespace sp
