// 2-D five-point stencil (fp32, one sweep) under a remap of tile ids.
//
// The paper lists "Stencil 2D" among its science kernels and re-orders its block grid so that blocks which share
// halo data run on the same chiplet's L2.  This is the same kind of workload for B200, sharing the remap library
// with the GEMM and the transpose:
//     out[i][j] = c_center * in[i][j] + c_neighbor * (in[i-1][j] + in[i+1][j] + in[i][j-1] + in[i][j+1])
// inside the grid, out = in on its rim.  The grid is cut into 64 x 128 tiles; persistent CTA b handles slots
// b, b + grid, ...; slot s works on tile slot_to_tile(s).
//
// Per tile: one TMA load of the tile plus its halo, 66 rows x 136 columns (the box starts 4 columns, i.e. 16 bytes,
// left of the tile: a TMA copy must start on a 16-byte boundary; out-of-range parts are filled with zeros and never
// used, because rim points copy their input), into a ring of three buffers.  Eight consumer warps take eight rows
// each: a lane owns four adjacent columns, keeps a three-row window in registers, gets its west / east neighbours
// from the adjacent lanes by shuffle (the outermost lanes read the halo columns), and writes 16 bytes per row into a
// staging slice of its warp (8 rows x 512 bytes, two per warp), which lane 0 then sends out with one TMA store.
// Memory bound: every input byte is read from HBM once (halos come from L2), every output byte written once.
#include <cuda.h>
#include <cuda_runtime.h>

#include "internal.h"
#include "ptx.cuh"

namespace sp {

constexpr int kStTileM = SP_STENCIL_TILE_M, kStTileN = SP_STENCIL_TILE_N;
constexpr int kStBoxRows = kStTileM + 2, kStBoxCols = kStTileN + 8;
constexpr uint32_t kStBoxBytes = kStBoxRows * kStBoxCols * 4;          // 35904
constexpr uint32_t kStBuf = (kStBoxBytes + 1023u) & ~1023u;             // buffers stay 1 KiB aligned
constexpr int kStStages = 3;     // measured: four to six buffers are no faster (row-major 6.31 TB/s with four, 6.40 with three);
constexpr int kStCtasPerSm = 1;  //   two or three CTAs per SM with fewer buffers each are 12-15 % slower (more tiles in flight
                                 //   at once, poorer DRAM page locality)
constexpr int kStConsumerWarps = 8;
constexpr int kStRowsPerWarp = kStTileM / kStConsumerWarps;
constexpr int kStThreads = 32 * (kStConsumerWarps + 1);
// Output: every consumer warp owns two staging slices of its 8 rows x 128 columns and sends a finished slice out with one
// TMA store (16-byte stores from registers reached 0.945 of the copy bandwidth in row-major order, 0.82-0.89 otherwise).
constexpr uint32_t kStOutSlice = kStRowsPerWarp * kStTileN * 4;                      // 4 KiB
constexpr uint32_t kStOutBytes = kStConsumerWarps * 2 * kStOutSlice;                 // 64 KiB
constexpr uint32_t kStSmem = kStStages * kStBuf + kStOutBytes + 1024 + 128;
static_assert(kStTileN == 128, "a lane owns four of the 128 columns of a tile row");

struct StencilArgs {
  const int32_t* perm;
  int32_t* status;
  float* out;
  int M, N;
  float c_center, c_neighbor;
  Sched sched;
};

enum : int { kRoleStencilLoad = 5, kRoleStencilCompute = 6 };

__device__ __forceinline__ float4 lds128(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}

__device__ __forceinline__ float lds32(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}

__global__ void __launch_bounds__(kStThreads, kStCtasPerSm)
stencil_kernel(const __grid_constant__ CUtensorMap tmIn, const __grid_constant__ CUtensorMap tmOut, const StencilArgs args) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t out_base = base + kStStages * kStBuf;
  const uint32_t bar_full = out_base + kStOutBytes, bar_empty = bar_full + 8 * kStStages;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int T = args.sched.T, Tn = args.sched.Tn;
  const int step = gridDim.x;
  auto tile_of = [&](int s) { return args.sched.use_table ? __ldg(args.perm + s) : slot_to_tile(args.sched, s); };

  if (tid == 0) {
    for (int i = 0; i < kStStages; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, kStConsumerWarps); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == kStConsumerWarps) {
    // ---------------------------------------------------------------- producer: whole warp in the loop, one lane issues
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int s = blockIdx.x; s < T && ok; s += step) {
      ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, args.status, (kRoleStencilLoad << 8) | 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const int t = tile_of(s);
      const int tm = t / Tn, tn = t - tm * Tn;
      if (elect_one()) {
        mbar_arrive_expect_tx(bar_full + 8 * stage, kStBoxBytes);
        tma_load_2d<1>(base + stage * kStBuf, &tmIn, tn * kStTileN - 4, tm * kStTileM - 1, bar_full + 8 * stage);
      }
      __syncwarp();
      if (++stage == kStStages) { stage = 0; phase ^= 1u; }
    }
    // every buffer handed out must have been released: no copy is in flight towards this CTA when it exits
    for (int i = 0; i < kStStages && ok; ++i) {
      ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, args.status, (kRoleStencilLoad << 8) | 2);
      ok = __all_sync(0xffffffffu, ok);
      if (++stage == kStStages) { stage = 0; phase ^= 1u; }
    }
    if (!ok) {
      const unsigned long long t0 = globaltimer();
      while (globaltimer() - t0 < 1000000ull) __nanosleep(1000);  // let copies in flight land
    }
    return;
  }

  // ------------------------------------------------------------------ consumers
  const float c0 = args.c_center, c1 = args.c_neighbor;
  const int r0 = warp * kStRowsPerWarp;            // first tile row of this warp
  int stage = 0;
  uint32_t phase = 0;
  bool ok = true;
  uint32_t parity = 0;                             // which of this warp's two output slices
  for (int s = blockIdx.x; s < T && ok; s += step) {
    ok = mbar_wait(bar_full + 8 * stage, phase, args.status, (kRoleStencilCompute << 8) | 1);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) break;
    // the store issued two tiles ago (lane 0's: bulk groups belong to a thread) has read the slice about to be refilled
    if (lane == 0) bulk_wait_read_1();
    __syncwarp();
    const uint32_t slice = out_base + ((uint32_t)warp * 2u + parity) * kStOutSlice + (uint32_t)lane * 16u;
    const int t = tile_of(s);
    const int tm = t / Tn, tn = t - tm * Tn;
    const int gj = tn * kStTileN + 4 * lane;       // first of this lane's four columns
    // box row b holds grid row tm * 64 + b - 1; box column c holds grid column tn * 128 + c - 4
    const uint32_t col = base + stage * kStBuf + (uint32_t)(4 + 4 * lane) * 4u;
    auto row_addr = [&](int b) { return col + (uint32_t)b * (kStBoxCols * 4u); };
    float4 up = lds128(row_addr(r0)), cur = lds128(row_addr(r0 + 1));
#pragma unroll
    for (int k = 0; k < kStRowsPerWarp; ++k) {
      const int b = r0 + k + 1;                    // box row of the output row
      const int gi = tm * kStTileM + r0 + k;
      const float4 down = lds128(row_addr(b + 1));
      float west = __shfl_up_sync(0xffffffffu, cur.w, 1), east = __shfl_down_sync(0xffffffffu, cur.x, 1);
      if (lane == 0) west = lds32(row_addr(b) - 4u);
      if (lane == 31) east = lds32(row_addr(b) + 16u);
      float4 o;
      o.x = fmaf(c1, (up.x + down.x) + (west + cur.y), c0 * cur.x);
      o.y = fmaf(c1, (up.y + down.y) + (cur.x + cur.z), c0 * cur.y);
      o.z = fmaf(c1, (up.z + down.z) + (cur.y + cur.w), c0 * cur.z);
      o.w = fmaf(c1, (up.w + down.w) + (cur.z + east), c0 * cur.w);
      if (gi == 0 || gi == args.M - 1) o = cur;    // the rim keeps its input
      if (gj == 0) o.x = cur.x;
      if (gj + 3 == args.N - 1) o.w = cur.w;
      // (points beyond the grid's edge are written too: the store below is clipped there)
      st_shared_16(slice + (uint32_t)k * (kStTileN * 4u), __float_as_uint(o.x), __float_as_uint(o.y), __float_as_uint(o.z),
                   __float_as_uint(o.w));
      up = cur;
      cur = down;
    }
    fence_async_smem();                            // the slice must be visible to the copy engine
    __syncwarp();
    if (lane == 0) {
      // relaxed: the input buffer only needs the warp's shared-memory reads to be over, and they are, their values
      // having been used
      mbar_arrive_relaxed(bar_empty + 8 * stage);
      const int gi0 = tm * kStTileM + r0;
      if (gi0 < args.M) tma_store_2d(&tmOut, slice, tn * kStTileN, gi0);   // lane 0: `slice` is the slice's first byte
      bulk_commit();
    }
    parity ^= 1u;
    if (++stage == kStStages) { stage = 0; phase ^= 1u; }
  }
  if (lane == 0) bulk_wait_all();
}

int launch_stencil(const void* in, void* out, int64_t M, int64_t N, float c_center, float c_neighbor, const Sched& sched,
                   const int32_t* perm_dev, int32_t* status_dev, cudaStream_t stream) {
  CUtensorMap tmIn, tmOut;
  int rc = make_map_plain(&tmIn, in, M, N, kStBoxRows, kStBoxCols);
  if (rc == SP_OK) rc = make_map_plain(&tmOut, out, M, N, kStRowsPerWarp, kStTileN);
  if (rc != SP_OK) return rc;
  static uint64_t configured = 0;   // one bit per device
  cudaError_t e;
  if (first_use_on_this_device(configured)) {
    e = cudaFuncSetAttribute(stencil_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStSmem);
    if (e != cudaSuccess) { configured = 0; set_error("cudaFuncSetAttribute failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
  }
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    set_error("cannot query the device");
    return SP_ERR_CUDA;
  }
  int64_t grid = (int64_t)sms * kStCtasPerSm;
  if (grid > sched.T) grid = sched.T;
  StencilArgs args;
  args.perm = perm_dev;
  args.status = status_dev;
  args.out = static_cast<float*>(out);
  args.M = (int)M; args.N = (int)N;
  args.c_center = c_center; args.c_neighbor = c_neighbor;
  args.sched = sched;
  stencil_kernel<<<(unsigned)grid, kStThreads, kStSmem, stream>>>(tmIn, tmOut, args);
  e = cudaGetLastError();
  if (e != cudaSuccess) { set_error("stencil launch failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
  return SP_OK;
}

}  // namespace sp
