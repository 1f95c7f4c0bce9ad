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
//   single pass     -- a block of whole rows (48 KiB where the row length allows, 64 KiB at most) is brought into shared
//                      memory once and read from there into registers once; maximum, exponentials, sum and the normalised
//                      values are all taken there, the results written back to the same buffer and sent out from it by
//                      one bulk copy.  Every byte crosses HBM once in each direction; the order of the row blocks has
//                      nothing left to improve.  Rows of up to 1792 elements are handled a warp per row (no meeting of
//                      warps at all), longer ones by two to twelve warps per row (two meetings per block), rows of more
//                      than 16384 elements by the two to eight CTAs of a thread-block cluster, which exchange their partial
//                      results through distributed shared memory.
//
// All kernels: persistent CTAs (one per SM), one producer warp that brings tiles into a ring of three 64 KiB buffers (a
// block of whole rows is contiguous in memory: one bulk copy; a 32 x 512 tile: two TMA boxes of 32 rows x 1 KiB;
// completion counted on an mbarrier) and, where a kernel has output, sends each buffer out again once the consumer warps
// have left their results in it (16-byte stores from the consumers' registers reached 0.89 of the copy bandwidth at
// 16384 x 16384, bulk stores 0.98); eight to fifteen consumer warps.  Every wait is bounded and reports into the status
// word like the other kernels.
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
// Long rows take up to 15 consumer warps: with two warps per scheduler the chain of shared-memory reads, exponentials and
// shuffles of a block is latency-bound and, for blocks of several rows, longer than the block's share of the memory time
// (rows of 4096: 5.2 TB/s with 8 warps).  16 warps with the producer leave 128 registers per thread.
constexpr int kSmBlockWarpsMax = 16;
constexpr int kSmMaxRows = 8;                            // single pass, long rows: room for the partials of a block (it has at most six rows)
constexpr int kSmWarpRowLimit = 1792;                    // single pass: rows up to this length are handled a warp per row
constexpr uint32_t kSmSmem = kSmStages * kSmStageBytes + 1024 /* alignment */ + 64 /* barriers */ + (2 * kSmMaxRows * kSmBlockWarpsMax + 4) * 4 + 4 * 8 + 4 * 8 * 8;
static_assert(kSmTileM * kSmTileN * 4 == kSmStageBytes, "a two-phase tile fills one buffer");
constexpr int kSmPhaseWarps = 16;                       // two-phase kernels: consumer warps
static_assert(kSmTileM % kSmPhaseWarps == 0, "the rows of a two-phase tile are shared out evenly");

struct SoftmaxArgs {
  const float* in;
  float* out;
  float2* partial;       // two-phase: [row][column chunk] = (maximum, sum of exp(x - maximum))
  const int32_t* perm;
  int32_t* status;
  int M, N;
  int rows_per_block;    // single pass: rows of one block (1..96); a block's rows are contiguous in memory
  int reverse;           // phase 2: slot s works on the tile of slot T - 1 - s
  int chunk;             // rows spread over a cluster: elements of a row per CTA (a multiple of 4)
  Sched sched;
};

enum : int { kRoleSoftmaxLoad = 7, kRoleSoftmaxCompute = 8 };
enum : int { kSmSinglePass = 0, kSmPhase1 = 1, kSmPhase2 = 2, kSmCluster = 3 };

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
__device__ __forceinline__ void sm_sts128(uint32_t addr, const float4& v) {
  asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
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
// Contiguous bytes from shared to global memory (both 16-byte aligned, size a multiple of 16), bulk-group completion.
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_release(uint32_t bar) {
  asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
template <int W>
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(32 * W) : "memory"); }
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
// The same over aligned groups of LPR lanes (LPR a power of two): every lane of a group gets its group's result.
template <int LPR>
__device__ __forceinline__ float group_max(float v) {
#pragma unroll
  for (int o = LPR / 2; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
template <int LPR>
__device__ __forceinline__ float group_sum(float v) {
#pragma unroll
  for (int o = LPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
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
  uint32_t xbar, xval;   // rows spread over a cluster: four exchange barriers, [4][8] pairs of floats (see softmax_cluster_kernel)
};
__device__ __forceinline__ SmLayout sm_layout(const uint8_t* smem_raw) {
  SmLayout l;
  l.base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  l.bar_full = l.base + kSmStages * kSmStageBytes;
  l.bar_empty = l.bar_full + 8 * kSmStages;
  l.red = l.bar_empty + 8 * kSmStages + 16;              // [2][kSmMaxRows][consumer warps] floats (long rows, single pass)
  l.fail_flag = l.red + 2 * kSmMaxRows * kSmBlockWarpsMax * 4;
  l.xbar = l.fail_flag + 8;
  l.xval = l.xbar + 4 * 8;
  return l;
}

// Rows and columns of tile t.  Two-phase: a Tm x Tn grid of 32 x 512 tiles; single pass: Tm x 1 blocks of whole rows.
template <int MODE>
__device__ __forceinline__ void sm_geometry(const SoftmaxArgs& a, int t, int& row0, int& nrows, int& col0, int& ncols) {
  if (MODE == kSmSinglePass) {
    row0 = t * a.rows_per_block; nrows = min(a.rows_per_block, a.M - row0); col0 = 0; ncols = a.N;
  } else if (MODE == kSmCluster) {       // one row per slot; this CTA's share of it
    row0 = t; nrows = 1; col0 = (int)cluster_ctarank() * a.chunk; ncols = max(0, min(a.chunk, a.N - col0));
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

__device__ __forceinline__ void sm_init(const SmLayout& l, int consumer_warps = kSmWarps) {
  if (threadIdx.x == 0) {
    sm_sts32(l.fail_flag, 0.f);
    for (int i = 0; i < kSmStages; ++i) { mbar_init(l.bar_full + 8 * i, 1); mbar_init(l.bar_empty + 8 * i, consumer_warps); }
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
__device__ __forceinline__ void sm_produce(const SoftmaxArgs& args, const SmLayout& l, const CUtensorMap* tm_in, const CUtensorMap* tm_out) {
  constexpr bool STORE = MODE != kSmPhase1;      // the first phase leaves only its partials, written by the consumers
  int stage = 0;
  uint32_t phase = 0;
  bool ok = true;
  const int lane = threadIdx.x & 31;
  // The consumers leave their results in the buffer they were given and hand it back only then; this warp sends the
  // block out with bulk copies (a block of whole rows is contiguous in the output as in the input: one copy; a tile:
  // its two boxes, clipped at the matrix edge), waits until they have read the buffer, and fills it again.  Measured
  // against 16-byte stores from the consumers' registers at 16384 x 16384: 6.36 against 5.77 TB/s.  One lane issues,
  // commits and waits: bulk groups belong to a thread.
  auto store_block = [&](int s_prev, int st) {
    int row0, nrows, col0, ncols;
    sm_geometry<MODE>(args, sm_tile_of<MODE>(args, s_prev), row0, nrows, col0, ncols);
    if (lane == 0) {
      const uint32_t src = l.base + st * kSmStageBytes;
      if (MODE == kSmSinglePass || MODE == kSmCluster) {
        if (ncols > 0) bulk_store(args.out + (size_t)row0 * args.N + col0, src, (uint32_t)nrows * (uint32_t)ncols * 4u);
      } else {
        tma_store_2d(tm_out, src, col0, row0);
        if (ncols > kSmBoxCols) tma_store_2d(tm_out, src + kSmBoxBytes, col0 + kSmBoxCols, row0);
      }
      bulk_commit();
      bulk_wait_read_0();
    }
    __syncwarp();
  };
  // slots of this CTA: its own index and stride, or its cluster's when a row is spread over a cluster
  const int first = MODE == kSmCluster ? (int)(blockIdx.x / cluster_nctarank()) : (int)blockIdx.x;
  const int step = MODE == kSmCluster ? (int)(gridDim.x / cluster_nctarank()) : (int)gridDim.x;
  int n_loaded = 0;
  for (int s = first; s < args.sched.T && ok; s += step, ++n_loaded) {
    ok = mbar_wait(l.bar_empty + 8 * stage, phase ^ 1u, args.status, (kRoleSoftmaxLoad << 8) | 1);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) break;
    if (STORE && n_loaded >= kSmStages) store_block(s - kSmStages * step, stage);
    int row0, nrows, col0, ncols;
    sm_geometry<MODE>(args, sm_tile_of<MODE>(args, s), row0, nrows, col0, ncols);
    const uint32_t full = l.bar_full + 8 * stage, dst = l.base + stage * kSmStageBytes;
    if (elect_one()) {
      if (MODE == kSmSinglePass || MODE == kSmCluster) {
        const uint32_t bytes = (uint32_t)nrows * (uint32_t)ncols * 4u;
        mbar_arrive_expect_tx(full, bytes);         // (a share of no columns: the phase completes by the arrival alone)
        if (bytes) bulk_load(dst, args.in + (size_t)row0 * args.N + col0, bytes, full);
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
    // the last blocks: block n_loaded - kSmStages + i went through this stage, if there was one
    const int j = n_loaded - kSmStages + i;
    if (STORE && ok && j >= 0) store_block(first + j * step, stage);
    if (++stage == kSmStages) { stage = 0; phase ^= 1u; }
  }
  if (STORE && lane == 0) bulk_wait_all();      // ... nor away from it
  if (!ok) {
    const unsigned long long t0 = globaltimer();
    while (globaltimer() - t0 < 1000000ull) __nanosleep(1000);
  }
}

// ------------------------------------------------------------------ single pass, long rows: G warps on every row
// A block has ROWS rows (fewer in the last block) and G * ROWS consumer warps; warp w works on slice w % G of row w / G and
// a lane owns 16-byte units (slice * 32 + lane) + 32 * G * k, k < UK, of that row.  So a thread reduces one row only, however
// many rows the block has: one warp reduction and G partials per phase (all warps on every row instead cost a reduction
// per row and thread, and blocks of four to seven rows ran a fifth to a third below those of one row).  The block is read
// from shared memory once and then lives in registers; the warps meet twice per block.
template <int UK, int G, int ROWS>
__global__ void __launch_bounds__(32 * (G * ROWS + 1), 1) softmax_block_kernel(const __grid_constant__ CUtensorMap tm_in, const __grid_constant__ CUtensorMap tm_out,
                                                                              const SoftmaxArgs args) {
  constexpr int W = G * ROWS;
  static_assert(W <= kSmBlockWarpsMax, "the partials of a block have room for kSmBlockWarpsMax warps");
  extern __shared__ uint8_t smem_raw[];
  const SmLayout l = sm_layout(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int N = args.N;
  const uint32_t row_pitch = (uint32_t)N * 4u;
  sm_init(l, W);
  if (warp == W) { sm_produce<kSmSinglePass>(args, l, &tm_in, &tm_out); return; }

  const int row = warp / G, slice = warp - row * G;
  const uint32_t red_max = l.red + (uint32_t)(row * G) * 4u, red_sum = red_max + (uint32_t)kSmBlockWarpsMax * 4u;
  int stage = 0;
  uint32_t phase = 0;
  const int nvec = N >> 2;
  for (int s = blockIdx.x; s < args.sched.T; s += gridDim.x) {
    bool ok = mbar_wait(l.bar_full + 8 * stage, phase, args.status, (kRoleSoftmaxCompute << 8) | 1);
    ok = __all_sync(0xffffffffu, ok);
    // The warps meet at named barriers below, so none may leave on its own: a warp whose wait gave up raises a flag,
    // goes through the first meeting empty-handed, and all of them leave together right after it.
    if (!ok && lane == 0) sm_sts32(l.fail_flag, 1.f);
    int row0, nrows, col0, ncols;
    sm_geometry<kSmSinglePass>(args, sm_tile_of<kSmSinglePass>(args, s), row0, nrows, col0, ncols);
    const bool mine = ok && row < nrows;
    const uint32_t base = l.base + stage * kSmStageBytes + (uint32_t)row * row_pitch;
    float4 v[UK];
    float acc = -INFINITY;
#pragma unroll
    for (int k = 0; k < UK; ++k) {
      const int i = slice * 32 + lane + 32 * G * k;
      if (mine && i < nvec) {
        v[k] = sm_lds128(base + (uint32_t)i * 16u);
        acc = fmaxf(acc, max4(v[k]));
      }
    }
    acc = warp_max(acc);
    if (lane == 0) sm_sts32(red_max + (uint32_t)slice * 4u, acc);
    consumer_sync<W>();
    if (sm_lds32(l.fail_flag) != 0.f) break;
    float big = -INFINITY;
#pragma unroll
    for (int g = 0; g < G; ++g) big = fmaxf(big, sm_lds32(red_max + (uint32_t)g * 4u));
    acc = 0.f;
#pragma unroll
    for (int k = 0; k < UK; ++k)
      if (mine && slice * 32 + lane + 32 * G * k < nvec) acc += exp4_sum(v[k], big);
    acc = warp_sum(acc);
    if (lane == 0) sm_sts32(red_sum + (uint32_t)slice * 4u, acc);
    consumer_sync<W>();
    // (the sums are read below by every warp before any of them can pass the next block's first meeting, after which
    // alone they are rewritten; the maxima were all read before the second meeting)
    if (mine) {
      float total = 0.f;
#pragma unroll
      for (int g = 0; g < G; ++g) total += sm_lds32(red_sum + (uint32_t)g * 4u);
      const float inv = 1.f / total;
#pragma unroll
      for (int k = 0; k < UK; ++k) {
        const int i = slice * 32 + lane + 32 * G * k;
        if (i < nvec) {
          float4 o = v[k];
          o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
          sm_sts128(base + (uint32_t)i * 16u, o);   // back to where it came from
        }
      }
    }
    // the results are in the buffer: make them visible to the copy engine, then hand the buffer to the producer warp
    fence_async_smem();
    __syncwarp();
    if (lane == 0) mbar_arrive_release(l.bar_empty + 8 * stage);
    if (++stage == kSmStages) { stage = 0; phase ^= 1u; }
  }
}

// ------------------------------------------------------------------ single pass, rows longer than a buffer: a cluster per row
// A row of up to CS x 16384 elements is spread over the CS CTAs of a thread-block cluster: CTA k brings elements
// [k * chunk, (k + 1) * chunk) of the row into its own ring.  One sweep and one exchange per row:
//   sweep    -- a thread reads its units of the share (G warps, UK units per lane), takes their maximum m_t, writes
//               exp(x - m_t) back in place and keeps (m_t, s_t = sum of those); pairs combine as (m, s) + (m', s') =
//               (M = max(m, m'), s exp(m - M) + s' exp(m' - M)): by shuffles within a warp, through shared memory across
//               the warps (one meeting of the consumer warps per row), and
//   exchange -- across the CTAs through distributed shared memory: one thread writes its CTA's pair into slot k of every
//               CTA of the cluster and arrives, with release at cluster scope, on that CTA's exchange barrier;
//   scaling  -- a thread waits on its own CTA's barrier (bounded, acquire at cluster scope), combines the CS pairs into
//               (M, S), and multiplies its units by exp(m_t - M) / S; the buffer then goes to the producer warp, which
//               sends it out.
// The scaling of a row is done after the sweep of the next one, so the exchange has a sweep's time to complete.  A long
// row crosses HBM once in each direction, where the two-phase form reads it twice.
// Exchange slots and barriers go round four sets: a CTA can publish row j + 3 while a peer still reads the pairs of row j
// (it needs nothing from that peer until it scales row j + 2), but row j + 4 only after the peer has published row
// j + 2, which the peer does after it has scaled row j.  No hardware cluster barrier inside the loop: every wait is
// bounded, so a CTA whose wait gave up leaves the loop, its peers' waits run out in turn, and all of them meet at the
// cluster barrier before the exit (shared memory of a CTA that has exited must not be written).
__device__ __forceinline__ void pair_combine(float& m, float& s, float m2, float s2) {
  const float M = fmaxf(m, m2);
  // a pair (-inf, 0) stands for "nothing": its share of the sum is 0, not exp(-inf + inf)
  s = (m == -INFINITY ? 0.f : s * exp_diff(m, M)) + (m2 == -INFINITY ? 0.f : s2 * exp_diff(m2, M));
  m = M;
}
template <int UK, int G, int CS>
__global__ void __launch_bounds__(32 * (G + 1), 1) softmax_cluster_kernel(const __grid_constant__ CUtensorMap tm_in, const __grid_constant__ CUtensorMap tm_out,
                                                                          const SoftmaxArgs args) {
  constexpr int W = G;
  extern __shared__ uint8_t smem_raw[];
  const SmLayout l = sm_layout(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  sm_init(l, W);
  if (tid == 0) {
    for (int i = 0; i < 4; ++i) mbar_init(l.xbar + 8 * i, CS);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // every CTA's barriers exist before any peer arrives on them
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");

  if (warp == W) {
    sm_produce<kSmCluster>(args, l, &tm_in, &tm_out);
  } else {
    const int first = (int)(blockIdx.x / CS), step = (int)(gridDim.x / CS);
    const int T = args.sched.T;
    int stage = 0;
    uint32_t phase = 0;
    // the row swept in the previous iteration, waiting to be scaled
    bool pending = false;
    int p_stage = 0, p_nvec = 0, p_it = 0;
    float p_mt = 0.f;
    int it = 0;
    for (int s = first;; s += step, ++it) {
      const bool have = s < T;
      if (!have && !pending) break;
      int c_nvec = 0;
      float mt = -INFINITY;
      if (have) {
        bool ok = mbar_wait(l.bar_full + 8 * stage, phase, args.status, (kRoleSoftmaxCompute << 8) | 1);
        ok = __all_sync(0xffffffffu, ok);
        // The warps meet below, so none may leave on its own: a warp whose wait gave up raises a flag, goes through the
        // meeting empty-handed, and all of them leave together right after it.
        if (!ok && lane == 0) sm_sts32(l.fail_flag, 1.f);
        int row0, nrows, col0, ncols;
        sm_geometry<kSmCluster>(args, sm_tile_of<kSmCluster>(args, s), row0, nrows, col0, ncols);
        c_nvec = ok ? ncols >> 2 : 0;
        const uint32_t base = l.base + stage * kSmStageBytes;
        float4 v[UK];
#pragma unroll
        for (int k = 0; k < UK; ++k) {
          const int i = warp * 32 + lane + 32 * G * k;
          if (i < c_nvec) {
            v[k] = sm_lds128(base + (uint32_t)i * 16u);
            mt = fmaxf(mt, max4(v[k]));
          }
        }
        float st = 0.f;
#pragma unroll
        for (int k = 0; k < UK; ++k) {
          const int i = warp * 32 + lane + 32 * G * k;
          if (i < c_nvec) {
            st += exp4_sum(v[k], mt);
            sm_sts128(base + (uint32_t)i * 16u, v[k]);      // exp(x - m_t) replaces x; scaled once (M, S) of the row are known
          }
        }
        float m = mt;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, st, o);
          pair_combine(m, st, m2, s2);
        }
        const uint32_t red = l.red + (uint32_t)((it & 1) * 2 * kSmBlockWarpsMax) * 4u;     // pairs of the warps, two sets
        if (lane == 0) { sm_sts32(red + (uint32_t)(2 * warp) * 4u, m); sm_sts32(red + (uint32_t)(2 * warp + 1) * 4u, st); }
        consumer_sync<W>();
        if (sm_lds32(l.fail_flag) != 0.f) break;
        if (tid == 0) {
          float cm = -INFINITY, cs = 0.f;
#pragma unroll
          for (int g = 0; g < G; ++g) pair_combine(cm, cs, sm_lds32(red + (uint32_t)(2 * g) * 4u), sm_lds32(red + (uint32_t)(2 * g + 1) * 4u));
          const uint32_t q = (uint32_t)it & 3u;
          const uint32_t slot = l.xval + (q * 8u + rank) * 8u, bar = l.xbar + q * 8u;
#pragma unroll
          for (uint32_t c = 0; c < (uint32_t)CS; ++c) {
            asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(mapa(slot, c)), "f"(cm), "f"(cs) : "memory");
            mbar_arrive_cluster(mapa(bar, c));
          }
        }
      }
      if (pending) {
        const uint32_t q = (uint32_t)p_it & 3u, xphase = (uint32_t)(p_it >> 2) & 1u;
        bool okx = mbar_wait_cluster_acquire(l.xbar + q * 8u, xphase, args.status, (kRoleSoftmaxCompute << 8) | 2);
        okx = __all_sync(0xffffffffu, okx);
        // (a warp whose wait gave up must not leave on its own either, or the others would wait for it at the next
        // row's meeting: it raises the flag and goes there with them; the status word is set by then, so that row's
        // wait for data returns at once)
        if (!okx && lane == 0) sm_sts32(l.fail_flag, 1.f);
        if (okx) {
          float M = -INFINITY, S = 0.f;
#pragma unroll
          for (int c = 0; c < CS; ++c)
            pair_combine(M, S, sm_lds32(l.xval + (q * 8u + (uint32_t)c) * 8u), sm_lds32(l.xval + (q * 8u + (uint32_t)c) * 8u + 4u));
          const float f = p_mt == -INFINITY ? 0.f : exp_diff(p_mt, M) / S;
          const uint32_t base = l.base + p_stage * kSmStageBytes;
#pragma unroll
          for (int k = 0; k < UK; ++k) {
            const int i = warp * 32 + lane + 32 * G * k;
            if (i < p_nvec) {
              float4 o = sm_lds128(base + (uint32_t)i * 16u);
              o.x *= f; o.y *= f; o.z *= f; o.w *= f;
              sm_sts128(base + (uint32_t)i * 16u, o);
            }
          }
          // the results are in the buffer: make them visible to the copy engine, then hand the buffer to the producer warp
          fence_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive_release(l.bar_empty + 8 * p_stage);
        }
      }
      pending = have;
      p_stage = stage; p_nvec = c_nvec; p_it = it; p_mt = mt;
      if (have && ++stage == kSmStages) { stage = 0; phase ^= 1u; }
    }
  }
  // no CTA leaves while a peer may still write to its shared memory or arrive on its barriers
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}

// ------------------------------------------------------------------ a warp per row: short rows (single pass), and the two phases
// A lane owns 16-byte units lane, lane + 32, ... (KW of them) of a row or row segment; a warp works on ROWS rows at a time
// (their loads and reductions interleave), rows warp, warp + W, ... of the tile (W consumer warps).
template <int MODE, int KW, int ROWS, int W, int LPR>
__global__ void __launch_bounds__(32 * (W + 1), 1) softmax_rows_kernel(const __grid_constant__ CUtensorMap tm_in, const __grid_constant__ CUtensorMap tm_out,
                                                                     const SoftmaxArgs args) {
  extern __shared__ uint8_t smem_raw[];
  const SmLayout l = sm_layout(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int N = args.N, Tn = args.sched.Tn;
  // LPR lanes work on a row (32 / LPR rows per warp at a time): very short rows would leave most lanes of a warp idle
  static_assert(LPR == 32 || MODE == kSmSinglePass, "the two-phase kernels put a whole warp on a row segment");
  constexpr int RPW = 32 / LPR;
  const int sl = lane & (LPR - 1), q = lane / LPR;
  sm_init(l, W);
  if (warp == W) { sm_produce<MODE>(args, l, &tm_in, &tm_out); return; }
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
    for (int rb = warp * RPW; rb < nrows; rb += W * RPW * ROWS) {
      float4 v[ROWS][KW];
      float m[ROWS];
      float2 part[ROWS];                       // phase 2: this lane's share of the row's partials, folded as they come
#pragma unroll
      for (int j = 0; j < ROWS; ++j) {
        const int r = rb + j * (W * RPW) + q;
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
            const int i = sl + LPR * k;
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
          big[j] = group_max<LPR>(m[j]);
          inv[j] = 0.f;
        }
      }
#pragma unroll
      for (int j = 0; j < ROWS; ++j) {
        const int r = rb + j * (W * RPW) + q;
        const bool live = r < nrows;          // with LPR < 32 the lanes of a warp hold different rows: no lane may skip a shuffle
        if (MODE == kSmPhase2) {
#pragma unroll
          for (int k = 0; k < KW; ++k) {
            const int i = sl + LPR * k;
            if (live && i < nvec) {
              float4 o = v[j][k];
              exp4_sum(o, big[j]);
              o.x *= inv[j]; o.y *= inv[j]; o.z *= inv[j]; o.w *= inv[j];
              sm_sts128(unit_addr(buf, r, i), o);       // results replace the inputs; the producer warp sends them out
            }
          }
        } else {
          float sum = 0.f;
#pragma unroll
          for (int k = 0; k < KW; ++k)
            if (live && sl + LPR * k < nvec) sum += exp4_sum(v[j][k], big[j]);
          sum = group_sum<LPR>(sum);
          if (!live) continue;
          if (MODE == kSmPhase1) {
            if (lane == 0) args.partial[(size_t)(row0 + r) * Tn + tn] = make_float2(big[j], sum);
          } else {
            const float sc = 1.f / sum;
#pragma unroll
            for (int k = 0; k < KW; ++k) {
              const int i = sl + LPR * k;
              if (i < nvec) {
                float4 o = v[j][k];
                o.x *= sc; o.y *= sc; o.z *= sc; o.w *= sc;
                sm_sts128(unit_addr(buf, r, i), o);
              }
            }
          }
        }
      }
    }
    // this warp is done with the buffer: its reads are over (first phase) or its rows hold their results, which must be
    // visible to the copy engine before the producer warp is told
    if (MODE != kSmPhase1) fence_async_smem();
    __syncwarp();
    if (lane == 0) {
      if (MODE == kSmPhase1) mbar_arrive_relaxed(l.bar_empty + 8 * stage);
      else mbar_arrive_release(l.bar_empty + 8 * stage);
    }
    if (++stage == kSmStages) { stage = 0; phase ^= 1u; }
  }
}

template <typename Kernel>
static int launch_one(Kernel kern, uint64_t& configured, const CUtensorMap& tm_in, const CUtensorMap& tm_out, const SoftmaxArgs& args,
                      int64_t tiles, cudaStream_t stream, int threads = kSmThreads) {
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
  kern<<<(unsigned)grid, threads, kSmSmem, stream>>>(tm_in, tm_out, args);
  e = cudaGetLastError();
  if (e != cudaSuccess) { set_error("softmax launch failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
  return SP_OK;
}

template <int UK, int G, int ROWS>
static int launch_block(const CUtensorMap& tm, const SoftmaxArgs& args, int64_t tiles, cudaStream_t stream) {
  static uint64_t configured = 0;   // per instantiation, one bit per device
  return launch_one(softmax_block_kernel<UK, G, ROWS>, configured, tm, tm, args, tiles, stream, 32 * (G * ROWS + 1));
}
// The instantiation whose UK covers `units` 16-byte units per row with G warps on a row: UK = ceil(units / (32 G)), from
// LO to HI for the row lengths that come with ROWS rows per block.
template <int G, int ROWS, int LO, int HI>
static int launch_block_for(int units, const CUtensorMap& tm, const SoftmaxArgs& args, int64_t tiles, cudaStream_t stream) {
  if constexpr (LO > HI) {
    set_error("softmax: no kernel for %d units per row with %d warps on each of %d rows", units, G, ROWS);
    return SP_ERR_UNSUPPORTED;
  } else {
    if ((units + 32 * G - 1) / (32 * G) <= LO) return launch_block<LO, G, ROWS>(tm, args, tiles, stream);
    return launch_block_for<G, ROWS, LO + 1, HI>(units, tm, args, tiles, stream);
  }
}
// A row per cluster of CS CTAs: as many clusters as can be resident at once (asked of the occupancy calculator), at most
// one per row.
template <int UK, int G, int CS>
static int launch_cluster(const CUtensorMap& tm, const SoftmaxArgs& args, int64_t rows, cudaStream_t stream) {
  static uint64_t configured = 0;
  static int clusters[64] = {};
  auto kern = softmax_cluster_kernel<UK, G, CS>;
  cudaError_t e;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { set_error("cannot query the device"); return SP_ERR_CUDA; }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(32 * (G + 1), 1, 1);
  cfg.dynamicSmemBytes = kSmSmem;
  cfg.stream = stream;
  cfg.attrs = attr; cfg.numAttrs = 1;
  if (first_use_on_this_device(configured)) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmSmem);
    if (e != cudaSuccess) { configured = 0; set_error("cudaFuncSetAttribute failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
    int sms = 0, n = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cfg.gridDim = dim3((unsigned)(sms / CS * CS), 1, 1);
    e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
    if (e != cudaSuccess || n < 1) {
      configured = 0; cudaGetLastError();
      set_error("no cluster of %d CTAs can be resident with this kernel (%s)", CS, e == cudaSuccess ? "0 active clusters" : cudaGetErrorString(e));
      return SP_ERR_UNSUPPORTED;
    }
    clusters[dev & 63] = n;
  }
  const int64_t n_clusters = rows < clusters[dev & 63] ? rows : clusters[dev & 63];
  cfg.gridDim = dim3((unsigned)(n_clusters * CS), 1, 1);
  e = cudaLaunchKernelEx(&cfg, kern, tm, tm, args);
  if (e != cudaSuccess) { set_error("softmax cluster launch failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
  return SP_OK;
}
template <int G, int CS, int LO, int HI>
static int launch_cluster_for(int units, const CUtensorMap& tm, const SoftmaxArgs& args, int64_t rows, cudaStream_t stream) {
  if constexpr (LO > HI) {
    set_error("softmax: no cluster kernel for %d units per share with %d warps", units, G);
    return SP_ERR_UNSUPPORTED;
  } else {
    if ((units + 32 * G - 1) / (32 * G) <= LO) return launch_cluster<LO, G, CS>(tm, args, rows, stream);
    return launch_cluster_for<G, CS, LO + 1, HI>(units, tm, args, rows, stream);
  }
}
template <int CS>
static int launch_cluster_share(int units, const CUtensorMap& tm, const SoftmaxArgs& args, int64_t rows, cudaStream_t stream) {
  // a share of 8196 to 16384 elements: twelve consumer warps (eight: 3-6 % slower, fifteen: the same)
  return launch_cluster_for<12, CS, 6, 11>(units, tm, args, rows, stream);
}

template <int MODE, int KW, int ROWS, int W = kSmWarps, int LPR = 32>
static int launch_rows(const CUtensorMap& tm, const CUtensorMap& tm_out, const SoftmaxArgs& args, int64_t tiles, cudaStream_t stream) {
  static uint64_t configured = 0;
  return launch_one(softmax_rows_kernel<MODE, KW, ROWS, W, LPR>, configured, tm, tm_out, args, tiles, stream, 32 * (W + 1));
}

// Single pass: rows of one block; 0 when a row does not fit a buffer.  A block is kept to 48 KiB where the row length
// allows: with three 64 KiB blocks in flight per SM the memory system is over-subscribed and delivers a tenth less
// (rows of 4096: 5.75 TB/s with blocks of four rows, 6.47 with three; four buffers of 48 KiB are no better than three).
// Long rows: floor(12288 / N) rows, at least one.  Short rows (a warp per row): a multiple of the eight consumer warps, 8 to 96.
int softmax_rows_per_block(int64_t N) {
  if (N * 4 > (int64_t)kSmStageBytes) return N <= 8 * (int64_t)(kSmStageBytes / 4) ? 1 : 0;   // a cluster of up to eight CTAs per row
  const int64_t r = 12288 / N;
  if (N > kSmWarpRowLimit) return r < 1 ? 1 : (int)r;
  const int64_t r8 = r / kSmWarps * kSmWarps;
  return (int)(r8 < kSmWarps ? kSmWarps : r8 > 96 ? 96 : r8);
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
  args.chunk = 0;
  args.sched = sched;
  const int64_t T = sched.T;
  CUtensorMap tm, tm_out;      // used by the two-phase kernels only; the single-pass kernels take them and ignore them
  memset(&tm, 0, sizeof tm);
  memset(&tm_out, 0, sizeof tm_out);
  if (mode != SP_SOFTMAX_SINGLE_PASS) {
    int rc = make_map_plain(&tm, in, M, N, kSmTileM, kSmBoxCols);
    if (rc == SP_OK) rc = make_map_plain(&tm_out, out, M, N, kSmTileM, kSmBoxCols);
    if (rc != SP_OK) return rc;
  }
  if (mode == SP_SOFTMAX_SINGLE_PASS && N * 4 > (int64_t)kSmStageBytes) {
    // the row does not fit one CTA's buffer: the fewest CTAs whose buffers hold it share it as a cluster (2 to 8; a cluster
    // need not be a power of two), in equal shares of a multiple of 4 elements: the larger the shares, the fewer exchanges
    // per byte (resident on B200: 148 CTAs in clusters of two, 135 of three, 132 of four and six, 130 of five, 120 of eight)
    // (clusters of seven cover 105 of 148 SMs, of eight 120: seven are never used)
    int cs = (int)((N + 16383) / 16384);
    if (cs == 7) cs = 8;
    args.chunk = (int)(((N + cs - 1) / cs + 3) / 4 * 4);
    const int units = args.chunk / 4;
    switch (cs) {
      case 2: return launch_cluster_share<2>(units, tm, args, M, stream);
      case 3: return launch_cluster_share<3>(units, tm, args, M, stream);
      case 4: return launch_cluster_share<4>(units, tm, args, M, stream);
      case 5: return launch_cluster_share<5>(units, tm, args, M, stream);
      case 6: return launch_cluster_share<6>(units, tm, args, M, stream);
      default: return launch_cluster_share<8>(units, tm, args, M, stream);
    }
  }
  if (mode == SP_SOFTMAX_SINGLE_PASS) {
    if (N <= kSmWarpRowLimit) {
      // 16-byte units per lane and row (N / 128, rounded up to what is instantiated), and how many rows a warp works on
      // together: two where a block has at least sixteen rows (N <= 768), else its one row
      if (N <= 64) return launch_rows<kSmSinglePass, 2, 2, kSmWarps, 8>(tm, tm_out, args, T, stream);
      if (N <= 128) return launch_rows<kSmSinglePass, 2, 2, kSmWarps, 16>(tm, tm_out, args, T, stream);
      if (N <= 256) return launch_rows<kSmSinglePass, 2, 2>(tm, tm_out, args, T, stream);
      if (N <= 512) return launch_rows<kSmSinglePass, 4, 2>(tm, tm_out, args, T, stream);
      if (N <= 768) return launch_rows<kSmSinglePass, 6, 2>(tm, tm_out, args, T, stream);
      if (N <= 1024) return launch_rows<kSmSinglePass, 8, 1>(tm, tm_out, args, T, stream);
      if (N <= 1536) return launch_rows<kSmSinglePass, 12, 1>(tm, tm_out, args, T, stream);
      return launch_rows<kSmSinglePass, 14, 1>(tm, tm_out, args, T, stream);
    }
    // Rows per block decide how many warps share a row; up to 15 consumer warps (with the
    // producer 16: four per scheduler, 128 registers each).  One row per block: 8 warps for the longest rows, 12 below
    // (measured: 6.37 against 5.80 TB/s at 16384, 6.08 against 6.60 at 12288).
    const int units = (int)(N / 4);
    switch (args.rows_per_block) {
      case 1: return units > 3072 ? launch_block_for<8, 1, 13, 16>(units, tm, args, T, stream)     // N in (12288, 16384]
                                  : launch_block_for<12, 1, 5, 8>(units, tm, args, T, stream);     // (6144, 12288]
      case 2: return launch_block_for<6, 2, 6, 8>(units, tm, args, T, stream);                      // (4096, 6144]
      case 3: return launch_block_for<4, 3, 7, 8>(units, tm, args, T, stream);                      // (3072, 4096]
      case 4: return launch_block_for<3, 4, 7, 8>(units, tm, args, T, stream);                      // (2457, 3072]
      case 5: return launch_block_for<3, 5, 6, 7>(units, tm, args, T, stream);                      // (2048, 2457]
      default: return launch_block_for<2, 6, 8, 8>(units, tm, args, T, stream);                     // (1792, 2048]
    }
  }
  // sixteen consumer warps, two rows of the tile each
  int rc = launch_rows<kSmPhase1, kSmTileN / 128, kSmTileM / kSmPhaseWarps, kSmPhaseWarps>(tm, tm_out, args, T, stream);
  if (rc != SP_OK) return rc;
  return launch_rows<kSmPhase2, kSmTileN / 128, kSmTileM / kSmPhaseWarps, kSmPhaseWarps>(tm, tm_out, args, T, stream);
}

}  // namespace sp
