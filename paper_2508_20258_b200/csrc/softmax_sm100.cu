// Row softmax (fp32) under a remap of tile ids, in the two forms the paper's softmax case study contrasts.
//
// The paper's kernel reduces every row in two phases (the maximum, then the exponentials and their sum) with the row cut
// into chunks that different blocks handle, and re-orders the blocks so that the chunks of a row meet in one chiplet's L2
// and are still there for the second phase.  Here:
//
//   two-phase form  -- the matrix is cut into 32 x 512 tiles ordered by the same remap library as the GEMM.  Phase 1
//                      (one launch) leaves, per tile and row, the partial maximum m and the partial sum of exp(x - m);
//                      phase 2 (a second launch) combines a row's partials (M = max m_c, S = sum s_c exp(m_c - M)),
//                      reads the tile again and writes exp(x - M) / S.  The second read comes from L2 when the tile is
//                      still there: phase 2 can walk the slots in the same order as phase 1 or backwards, starting with
//                      what phase 1 touched last.
//   single pass     -- a block of whole rows (64 KiB at most) is brought into shared memory once and read from there into
//                      registers once; maximum, exponentials, sum and the normalised values are all taken there.  Every
//                      byte crosses HBM once in each direction; the order of the row blocks has nothing left to improve.
//                      Rows of up to 2048 elements are handled a warp per row (no meeting of warps at all), longer ones by
//                      all eight warps together (two meetings per block).
//
// All kernels: persistent CTAs (one per SM), one producer warp that brings tiles into a ring of three 64 KiB buffers (a
// block of whole rows is contiguous in memory: one bulk copy; a 32 x 512 tile: two TMA boxes of 32 rows x 1 KiB;
// completion counted on an mbarrier), eight consumer warps, 16-byte streaming stores.  Every wait is bounded and reports into the status word like the other kernels.
#include <cuda.h>
#include <cuda_runtime.h>
#include <string.h>

#include "internal.h"
#include "ptx.cuh"

namespace sp {

constexpr int kSmTileM = SP_SOFTMAX_TILE_M, kSmTileN = SP_SOFTMAX_TILE_N;
constexpr uint32_t kSmStageBytes = 65536;
constexpr int kSmStages = 3;
constexpr int kSmWarps = 8;                              // consumer warps
constexpr int kSmThreads = 32 * (kSmWarps + 1);
constexpr int kSmMaxRows = 8;                            // single pass, long rows: rows per block
constexpr int kSmWarpRowLimit = 2048;                    // single pass: rows up to this length are handled a warp per row
constexpr uint32_t kSmSmem = kSmStages * kSmStageBytes + 1024 /* alignment */ + 64 /* barriers */ + (2 * kSmMaxRows * kSmWarps + 4) * 4;
static_assert(kSmTileM * kSmTileN * 4 == kSmStageBytes, "a two-phase tile fills one buffer");
static_assert(kSmTileM == 4 * kSmWarps, "a warp takes four rows of a two-phase tile");

struct SoftmaxArgs {
  const float* in;
  float* out;
  float2* partial;       // two-phase: [row][column chunk] = (maximum, sum of exp(x - maximum))
  const int32_t* perm;
  int32_t* status;
  int M, N;
  int rows_per_block;    // single pass: rows of one block (1..32); a block's rows are contiguous in memory
  int reverse;           // phase 2: slot s works on the tile of slot T - 1 - s
  Sched sched;
};

enum : int { kRoleSoftmaxLoad = 7, kRoleSoftmaxCompute = 8 };
enum : int { kSmSinglePass = 0, kSmPhase1 = 1, kSmPhase2 = 2 };

__device__ __forceinline__ float4 sm_lds128(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ float sm_lds32(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sm_sts32(uint32_t addr, float v) {
  asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
// Contiguous bytes from global to shared memory (both 16-byte aligned, size a multiple of 16); completion is counted
// in bytes on the mbarrier.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(32 * kSmWarps) : "memory"); }
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// exp(a - b) for a <= b, through the hardware's 2^x: the difference is rounded once, the product with log2(e) once
__device__ __forceinline__ float exp_diff(float a, float b) { return exp2f((a - b) * 1.4426950408889634f); }
__device__ __forceinline__ float max4(const float4& v) { return fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)); }
__device__ __forceinline__ float exp4_sum(float4& v, float big) {   // v <- exp(v - big); returns the sum of the four
  v.x = exp_diff(v.x, big); v.y = exp_diff(v.y, big); v.z = exp_diff(v.z, big); v.w = exp_diff(v.w, big);
  return (v.x + v.y) + (v.z + v.w);
}

struct SmLayout {
  uint32_t base, bar_full, bar_empty, red, fail_flag;
};
__device__ __forceinline__ SmLayout sm_layout(const uint8_t* smem_raw) {
  SmLayout l;
  l.base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  l.bar_full = l.base + kSmStages * kSmStageBytes;
  l.bar_empty = l.bar_full + 8 * kSmStages;
  l.red = l.bar_empty + 8 * kSmStages + 16;              // [2][kSmMaxRows][kSmWarps] floats (long rows, single pass)
  l.fail_flag = l.red + 2 * kSmMaxRows * kSmWarps * 4;
  return l;
}

// Rows and columns of tile t.  Two-phase: a Tm x Tn grid of 32 x 512 tiles; single pass: Tm x 1 blocks of whole rows.
template <int MODE>
__device__ __forceinline__ void sm_geometry(const SoftmaxArgs& a, int t, int& row0, int& nrows, int& col0, int& ncols) {
  if (MODE == kSmSinglePass) {
    row0 = t * a.rows_per_block; nrows = min(a.rows_per_block, a.M - row0); col0 = 0; ncols = a.N;
  } else {
    const int Tn = a.sched.Tn, tm = t / Tn, tn = t - tm * Tn;
    row0 = tm * kSmTileM; nrows = min(kSmTileM, a.M - row0); col0 = tn * kSmTileN; ncols = min(kSmTileN, a.N - col0);
  }
}
template <int MODE>
__device__ __forceinline__ int sm_tile_of(const SoftmaxArgs& a, int s) {
  if (MODE == kSmPhase2 && a.reverse) s = a.sched.T - 1 - s;
  return a.sched.use_table ? __ldg(a.perm + s) : slot_to_tile(a.sched, s);
}

__device__ __forceinline__ void sm_init(const SmLayout& l) {
  if (threadIdx.x == 0) {
    sm_sts32(l.fail_flag, 0.f);
    for (int i = 0; i < kSmStages; ++i) { mbar_init(l.bar_full + 8 * i, 1); mbar_init(l.bar_empty + 8 * i, kSmWarps); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
}

constexpr int kSmBoxCols = 256;                                         // a TMA box is at most 256 elements wide
constexpr uint32_t kSmBoxBytes = kSmTileM * kSmBoxCols * 4;             // 32 KiB: half a two-phase tile

// Producer warp: whole warp in the loop, one elected lane issues.  Single pass: the block's rows are contiguous, one bulk
// copy brings them all.  Two-phase: the tile comes as two boxes of 32 rows x 256 columns (parts outside the matrix are
// filled with zeros and never used; a box wholly outside is not requested).
template <int MODE>
__device__ __forceinline__ void sm_produce(const SoftmaxArgs& args, const SmLayout& l, const CUtensorMap* tm_in) {
  int stage = 0;
  uint32_t phase = 0;
  bool ok = true;
  for (int s = blockIdx.x; s < args.sched.T && ok; s += gridDim.x) {
    ok = mbar_wait(l.bar_empty + 8 * stage, phase ^ 1u, args.status, (kRoleSoftmaxLoad << 8) | 1);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) break;
    int row0, nrows, col0, ncols;
    sm_geometry<MODE>(args, sm_tile_of<MODE>(args, s), row0, nrows, col0, ncols);
    const uint32_t full = l.bar_full + 8 * stage, dst = l.base + stage * kSmStageBytes;
    if (elect_one()) {
      if (MODE == kSmSinglePass) {
        const uint32_t bytes = (uint32_t)nrows * (uint32_t)ncols * 4u;
        mbar_arrive_expect_tx(full, bytes);
        bulk_load(dst, args.in + (size_t)row0 * args.N, bytes, full);
      } else {
        const int boxes = ncols > kSmBoxCols ? 2 : 1;
        mbar_arrive_expect_tx(full, boxes * kSmBoxBytes);
        tma_load_2d<1>(dst, tm_in, col0, row0, full);
        if (boxes == 2) tma_load_2d<1>(dst + kSmBoxBytes, tm_in, col0 + kSmBoxCols, row0, full);
      }
    }
    __syncwarp();
    if (++stage == kSmStages) { stage = 0; phase ^= 1u; }
  }
  for (int i = 0; i < kSmStages && ok; ++i) {   // no copy may still be in flight towards this CTA when it exits
    ok = mbar_wait(l.bar_empty + 8 * stage, phase ^ 1u, args.status, (kRoleSoftmaxLoad << 8) | 2);
    ok = __all_sync(0xffffffffu, ok);
    if (++stage == kSmStages) { stage = 0; phase ^= 1u; }
  }
  if (!ok) {
    const unsigned long long t0 = globaltimer();
    while (globaltimer() - t0 < 1000000ull) __nanosleep(1000);
  }
}

// ------------------------------------------------------------------ single pass, long rows: all warps on every row
// KK = 16-byte units of a row per thread (ceil(N / 1024)), RMAX = the most rows a block can have at that KK.
template <int KK, int RMAX>
__global__ void __launch_bounds__(kSmThreads, 1) softmax_block_kernel(const __grid_constant__ CUtensorMap tm_in, const SoftmaxArgs args) {
  extern __shared__ uint8_t smem_raw[];
  const SmLayout l = sm_layout(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int N = args.N;
  const uint32_t row_pitch = (uint32_t)N * 4u;
  sm_init(l);
  if (warp == kSmWarps) { sm_produce<kSmSinglePass>(args, l, &tm_in); return; }

  int stage = 0;
  uint32_t phase = 0;
  const int nvec = N >> 2;
  for (int s = blockIdx.x; s < args.sched.T; s += gridDim.x) {
    bool ok = mbar_wait(l.bar_full + 8 * stage, phase, args.status, (kRoleSoftmaxCompute << 8) | 1);
    ok = __all_sync(0xffffffffu, ok);
    // The eight warps meet at named barriers below, so none may leave on its own: a warp whose wait gave up raises a
    // flag, goes through the first meeting empty-handed, and all of them leave together right after it.
    if (!ok && lane == 0) sm_sts32(l.fail_flag, 1.f);
    int row0, nrows, col0, ncols;
    sm_geometry<kSmSinglePass>(args, sm_tile_of<kSmSinglePass>(args, s), row0, nrows, col0, ncols);
    const uint32_t buf = l.base + stage * kSmStageBytes;
    // A thread owns 16-byte units tid, tid + 256, ... of each row.  The block is read from shared memory once and then
    // lives in registers (RMAX rows x KK units per thread, at most 21 units); the reductions of the block's rows are
    // batched: two meetings per block, not per row.
    float4 v[RMAX][KK];
    float acc[RMAX];
#pragma unroll
    for (int r = 0; r < RMAX; ++r) {
      acc[r] = -INFINITY;
#pragma unroll
      for (int k = 0; k < KK; ++k) {
        const int i = tid + 32 * kSmWarps * k;
        if (ok && r < nrows && i < nvec) {
          v[r][k] = sm_lds128(buf + (uint32_t)r * row_pitch + (uint32_t)i * 16u);
          acc[r] = fmaxf(acc[r], max4(v[r][k]));
        }
      }
      acc[r] = warp_max(acc[r]);
      if (lane == 0) sm_sts32(l.red + (uint32_t)(r * kSmWarps + warp) * 4u, acc[r]);
    }
    __syncwarp();
    if (lane == 0) mbar_arrive_relaxed(l.bar_empty + 8 * stage);   // the buffer has been read: the next copy may come
    consumer_sync();
    if (sm_lds32(l.fail_flag) != 0.f) break;
#pragma unroll
    for (int r = 0; r < RMAX; ++r) {
      float big = -INFINITY;
#pragma unroll
      for (int w = 0; w < kSmWarps; ++w) big = fmaxf(big, sm_lds32(l.red + (uint32_t)(r * kSmWarps + w) * 4u));
      acc[r] = 0.f;
#pragma unroll
      for (int k = 0; k < KK; ++k)
        if (r < nrows && tid + 32 * kSmWarps * k < nvec) acc[r] += exp4_sum(v[r][k], big);
      acc[r] = warp_sum(acc[r]);
      if (lane == 0) sm_sts32(l.red + (uint32_t)((kSmMaxRows + r) * kSmWarps + warp) * 4u, acc[r]);
    }
    consumer_sync();
    // (the sums are read below by every warp before any of them can pass the next block's first meeting, after which
    // alone they are rewritten; the maxima were all read before the second meeting)
#pragma unroll
    for (int r = 0; r < RMAX; ++r) {
      if (r < nrows) {
        float total = 0.f;
#pragma unroll
        for (int w = 0; w < kSmWarps; ++w) total += sm_lds32(l.red + (uint32_t)((kSmMaxRows + r) * kSmWarps + w) * 4u);
        const float inv = 1.f / total;
        float4* dst = reinterpret_cast<float4*>(args.out + (size_t)(row0 + r) * N);
#pragma unroll
        for (int k = 0; k < KK; ++k) {
          const int i = tid + 32 * kSmWarps * k;
          if (i < nvec) {
            float4 o = v[r][k];
            o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
            __stcs(dst + i, o);
          }
        }
      }
    }
    if (++stage == kSmStages) { stage = 0; phase ^= 1u; }
  }
}

// ------------------------------------------------------------------ a warp per row: short rows (single pass), and the two phases
// A lane owns 16-byte units lane, lane + 32, ... (KW of them) of a row or row segment; a warp works on ROWS rows at a time
// (their loads and reductions interleave), rows warp, warp + 8, ... of the tile.
template <int MODE, int KW, int ROWS>
__global__ void __launch_bounds__(kSmThreads, 1) softmax_rows_kernel(const __grid_constant__ CUtensorMap tm_in, const SoftmaxArgs args) {
  extern __shared__ uint8_t smem_raw[];
  const SmLayout l = sm_layout(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int N = args.N, Tn = args.sched.Tn;
  sm_init(l);
  if (warp == kSmWarps) { sm_produce<MODE>(args, l, &tm_in); return; }
  // 16-byte unit i of row r of a buffer: rows of N elements back to back (single pass), or two boxes of 32 rows x 1 KiB
  auto unit_addr = [&](uint32_t buf, int r, int i) -> uint32_t {
    if (MODE == kSmSinglePass) return buf + ((uint32_t)r * (uint32_t)N + (uint32_t)i * 4u) * 4u;
    return buf + (uint32_t)(i >> 6) * kSmBoxBytes + (uint32_t)r * (kSmBoxCols * 4u) + (uint32_t)(i & 63) * 16u;
  };

  int stage = 0;
  uint32_t phase = 0;
  for (int s = blockIdx.x; s < args.sched.T; s += gridDim.x) {
    bool ok = mbar_wait(l.bar_full + 8 * stage, phase, args.status, (kRoleSoftmaxCompute << 8) | 1);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) break;
    int row0, nrows, col0, ncols;
    sm_geometry<MODE>(args, sm_tile_of<MODE>(args, s), row0, nrows, col0, ncols);
    const uint32_t buf = l.base + stage * kSmStageBytes;
    const int nvec = ncols >> 2;
    const int tn = col0 / kSmTileN;
    for (int rb = warp; rb < nrows; rb += kSmWarps * ROWS) {
      float4 v[ROWS][KW];
      float m[ROWS];
      float2 part[ROWS];                       // phase 2: this lane's share of the row's partials, folded as they come
#pragma unroll
      for (int j = 0; j < ROWS; ++j) {
        const int r = rb + j * kSmWarps;
        m[j] = -INFINITY;
        part[j] = make_float2(-INFINITY, 0.f);
        if (r < nrows) {
          if (MODE == kSmPhase2) {
            // the row's partials from every column chunk: maximum of the maxima, sums rescaled to it (a lane folds
            // the chunks lane, lane + 32, ... first; the lanes are combined below)
            const float2* p = args.partial + (size_t)(row0 + r) * Tn;
            for (int c = lane; c < Tn; c += 32) {
              const float2 q = __ldcg(p + c);
              const float nm = fmaxf(part[j].x, q.x);
              part[j].y = part[j].y * exp_diff(part[j].x, nm) + q.y * exp_diff(q.x, nm);
              part[j].x = nm;
            }
          }
#pragma unroll
          for (int k = 0; k < KW; ++k) {
            const int i = lane + 32 * k;
            if (i < nvec) {
              v[j][k] = sm_lds128(unit_addr(buf, r, i));
              m[j] = fmaxf(m[j], max4(v[j][k]));
            }
          }
        }
      }
      float big[ROWS], inv[ROWS];
#pragma unroll
      for (int j = 0; j < ROWS; ++j) {
        if (MODE == kSmPhase2) {
          big[j] = warp_max(part[j].x);
          // a lane without a chunk holds (-inf, 0): its exponential is 0 and so is its share of the sum
          inv[j] = 1.f / warp_sum(part[j].x == -INFINITY ? 0.f : part[j].y * exp_diff(part[j].x, big[j]));
        } else {
          big[j] = warp_max(m[j]);
          inv[j] = 0.f;
        }
      }
#pragma unroll
      for (int j = 0; j < ROWS; ++j) {
        const int r = rb + j * kSmWarps;
        if (r >= nrows) continue;
        if (MODE == kSmPhase2) {
          float4* dst = reinterpret_cast<float4*>(args.out + (size_t)(row0 + r) * N + col0);
#pragma unroll
          for (int k = 0; k < KW; ++k) {
            const int i = lane + 32 * k;
            if (i < nvec) {
              float4 o = v[j][k];
              exp4_sum(o, big[j]);
              o.x *= inv[j]; o.y *= inv[j]; o.z *= inv[j]; o.w *= inv[j];
              __stcs(dst + i, o);
            }
          }
        } else {
          float sum = 0.f;
#pragma unroll
          for (int k = 0; k < KW; ++k)
            if (lane + 32 * k < nvec) sum += exp4_sum(v[j][k], big[j]);
          sum = warp_sum(sum);
          if (MODE == kSmPhase1) {
            if (lane == 0) args.partial[(size_t)(row0 + r) * Tn + tn] = make_float2(big[j], sum);
          } else {
            const float sc = 1.f / sum;
            float4* dst = reinterpret_cast<float4*>(args.out + (size_t)(row0 + r) * N);
#pragma unroll
            for (int k = 0; k < KW; ++k) {
              const int i = lane + 32 * k;
              if (i < nvec) {
                float4 o = v[j][k];
                o.x *= sc; o.y *= sc; o.z *= sc; o.w *= sc;
                __stcs(dst + i, o);
              }
            }
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive_relaxed(l.bar_empty + 8 * stage);   // this warp's shared-memory reads of the buffer are over
    if (++stage == kSmStages) { stage = 0; phase ^= 1u; }
  }
}

template <typename Kernel>
static int launch_one(Kernel kern, uint64_t& configured, const CUtensorMap& tm_in, const SoftmaxArgs& args, int64_t tiles,
                      cudaStream_t stream) {
  cudaError_t e;
  if (first_use_on_this_device(configured)) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmSmem);
    if (e != cudaSuccess) { configured = 0; set_error("cudaFuncSetAttribute failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
  }
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    set_error("cannot query the device");
    return SP_ERR_CUDA;
  }
  const int64_t grid = tiles < sms ? tiles : sms;
  kern<<<(unsigned)grid, kSmThreads, kSmSmem, stream>>>(tm_in, args);
  e = cudaGetLastError();
  if (e != cudaSuccess) { set_error("softmax launch failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
  return SP_OK;
}

template <int KK, int RMAX>
static int launch_block(const CUtensorMap& tm, const SoftmaxArgs& args, int64_t tiles, cudaStream_t stream) {
  static uint64_t configured = 0;   // per instantiation, one bit per device
  return launch_one(softmax_block_kernel<KK, RMAX>, configured, tm, args, tiles, stream);
}
template <int MODE, int KW, int ROWS>
static int launch_rows(const CUtensorMap& tm, const SoftmaxArgs& args, int64_t tiles, cudaStream_t stream) {
  static uint64_t configured = 0;
  return launch_one(softmax_rows_kernel<MODE, KW, ROWS>, configured, tm, args, tiles, stream);
}

// Single pass: rows of one block.  A block fills at most one 64 KiB buffer; short rows (a warp per row) come up to 32 to a
// block (one copy per lane of the producer warp), long rows up to 8.  0 when a row does not fit a buffer.
int softmax_rows_per_block(int64_t N) {
  const int64_t fit = (int64_t)kSmStageBytes / (N * 4);
  const int64_t cap = N <= kSmWarpRowLimit ? 32 : kSmMaxRows;
  return fit < 1 ? 0 : (int)(fit > cap ? cap : fit);
}

int launch_softmax(const void* in, void* out, int64_t M, int64_t N, int mode, const Sched& sched, const int32_t* perm_dev,
                   float* partial_dev, int32_t* status_dev, cudaStream_t stream) {
  SoftmaxArgs args;
  args.in = static_cast<const float*>(in);
  args.out = static_cast<float*>(out);
  args.partial = reinterpret_cast<float2*>(partial_dev);
  args.perm = perm_dev;
  args.status = status_dev;
  args.M = (int)M; args.N = (int)N;
  args.rows_per_block = mode == SP_SOFTMAX_SINGLE_PASS ? softmax_rows_per_block(N) : 0;
  args.reverse = mode == SP_SOFTMAX_TWO_PHASE_REVERSED ? 1 : 0;
  args.sched = sched;
  const int64_t T = sched.T;
  CUtensorMap tm;      // used by the two-phase kernels only; the single-pass kernels take it and ignore it
  memset(&tm, 0, sizeof tm);
  if (mode != SP_SOFTMAX_SINGLE_PASS) {
    const int rc = make_map_plain(&tm, in, M, N, kSmTileM, kSmBoxCols);
    if (rc != SP_OK) return rc;
  }
  if (mode == SP_SOFTMAX_SINGLE_PASS) {
    if (N <= kSmWarpRowLimit) {
      // 16-byte units per lane and row: N / 128 rounded up to a power of two; two rows of a warp in flight together
      if (N <= 256) return launch_rows<kSmSinglePass, 2, 2>(tm, args, T, stream);
      if (N <= 512) return launch_rows<kSmSinglePass, 4, 2>(tm, args, T, stream);
      if (N <= 1024) return launch_rows<kSmSinglePass, 8, 2>(tm, args, T, stream);
      return launch_rows<kSmSinglePass, 16, 2>(tm, args, T, stream);
    }
    // 16-byte units per thread and row, and the most rows a block has at that width (rows x N x 4 <= 64 KiB, <= 8)
    switch ((int)((N / 4 + 32 * kSmWarps - 1) / (32 * kSmWarps))) {
      case 3: return launch_block<3, 7>(tm, args, T, stream);
      case 4: return launch_block<4, 5>(tm, args, T, stream);
      case 5: return launch_block<5, 3>(tm, args, T, stream);
      case 6: return launch_block<6, 3>(tm, args, T, stream);
      case 7: return launch_block<7, 2>(tm, args, T, stream);
      case 8: return launch_block<8, 2>(tm, args, T, stream);
      case 9: return launch_block<9, 1>(tm, args, T, stream);
      case 10: return launch_block<10, 1>(tm, args, T, stream);
      case 11: return launch_block<11, 1>(tm, args, T, stream);
      case 12: return launch_block<12, 1>(tm, args, T, stream);
      case 13: return launch_block<13, 1>(tm, args, T, stream);
      case 14: return launch_block<14, 1>(tm, args, T, stream);
      case 15: return launch_block<15, 1>(tm, args, T, stream);
      default: return launch_block<16, 1>(tm, args, T, stream);
    }
  }
  int rc = launch_rows<kSmPhase1, kSmTileN / 128, 4>(tm, args, T, stream);
  if (rc != SP_OK) return rc;
  return launch_rows<kSmPhase2, kSmTileN / 128, 4>(tm, args, T, stream);
}

}  // namespace sp
