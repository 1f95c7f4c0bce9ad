// Tiled transpose of a matrix of 16-bit elements under a remap of tile ids.
//
// The paper's largest win is a transpose kernel whose tile grid is re-ordered so that both
// the reads and the transposed writes stay local to one chiplet's L2.  This is the same
// workload for B200, sharing the remap library with the GEMM: out (N x M) = in (M x N)^T,
// cut into 64 x 64 tiles; persistent CTA b handles slots b, b + grid, ...; slot s works on
// tile slot_to_tile(s).
//
// Per tile: one TMA load (64 rows x 128 bytes, 128-byte swizzle) into a ring of input
// buffers; the two warps transpose 8 x 8 blocks with ldmatrix.trans / stmatrix (both free of
// bank conflicts under the swizzle) into an output buffer; one TMA store.  Memory bound:
// every byte is read once and written once.
#include <cuda.h>
#include <cuda_runtime.h>

#include "internal.h"
#include "ptx.cuh"

namespace sp {

constexpr int kTrTile = 64;                 // elements per tile side
constexpr int kTrThreads = 64;
constexpr int kTrIn = 3, kTrOut = 3;        // input ring, output ring
constexpr uint32_t kTrBuf = kTrTile * kTrTile * 2;
constexpr uint32_t kTrSmem = (kTrIn + kTrOut) * kTrBuf + 1024 + 64;
constexpr int kTrCtasPerSm = 4;

struct TransposeArgs {
  const int32_t* perm;
  int32_t* status;
  Sched sched;
};

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}

__device__ __forceinline__ void stmatrix_x4(uint32_t addr, const uint32_t (&r)[4]) {
  asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(r[0]), "r"(r[1]),
               "r"(r[2]), "r"(r[3])
               : "memory");
}

__global__ void __launch_bounds__(kTrThreads, kTrCtasPerSm)
transpose_kernel(const __grid_constant__ CUtensorMap tmIn, const __grid_constant__ CUtensorMap tmOut,
                 const TransposeArgs args) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t in_base = base, out_base = base + kTrIn * kTrBuf, bar_full = out_base + kTrOut * kTrBuf;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int T = args.sched.T, Tn = args.sched.Tn;
  const int step = gridDim.x;

  auto tile_of = [&](int s) { return args.sched.use_table ? __ldg(args.perm + s) : slot_to_tile(args.sched, s); };
  auto issue_load = [&](int s, int stage) {       // tile of slot s into input buffer `stage`
    const int t = tile_of(s);
    const int tm = t / Tn, tn = t - tm * Tn;
    mbar_arrive_expect_tx(bar_full + 8 * stage, kTrBuf);
    tma_load_2d<1>(in_base + stage * kTrBuf, &tmIn, tn * kTrTile, tm * kTrTile, bar_full + 8 * stage);
  };

  if (tid == 0) {
    for (int i = 0; i < kTrIn; ++i) mbar_init(bar_full + 8 * i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (tid == 0) {
    for (int i = 0; i < kTrIn; ++i) {
      const int s = blockIdx.x + i * step;
      if (s < T) issue_load(s, i);
    }
  }

  // this lane's row inside each of the four 8 x 8 blocks an ldmatrix / stmatrix handles
  const int k = lane >> 3, j = lane & 7;
  bool ok = true;
  int it = 0;
  for (int s = blockIdx.x; s < T; s += step, ++it) {
    const int stage = it % kTrIn, obuf = it % kTrOut;
    const uint32_t phase = (uint32_t)(it / kTrIn) & 1u;
    ok = mbar_wait(bar_full + 8 * stage, phase, args.status, (4 << 8) | 1);
    if (!__syncthreads_and(ok)) break;
    const uint32_t src = in_base + stage * kTrBuf, dst = out_base + obuf * kTrBuf;
#pragma unroll
    for (int q4 = 0; q4 < 8; ++q4) {
      const int q = warp * 32 + q4 * 4 + k;       // block index: rows 8a.., 16-byte unit b of the input tile
      const int a = q >> 3, b = q & 7;
      uint32_t r[4];
      ldmatrix_x4_trans(src + (uint32_t)((8 * a + j) * 128 + ((b ^ j) << 4)), r);
      stmatrix_x4(dst + (uint32_t)((8 * b + j) * 128 + ((a ^ j) << 4)), r);
    }
    fence_async_smem();
    if (tid == 0) bulk_wait_read_1();             // the store issued two tiles ago has read its buffer
    __syncthreads();
    if (tid == 0) {
      const int t = tile_of(s);
      const int tm = t / Tn, tn = t - tm * Tn;
      tma_store_2d(&tmOut, dst, tm * kTrTile, tn * kTrTile);
      bulk_commit();
      const int nxt = s + kTrIn * step;           // refill the input buffer everybody has finished reading
      if (nxt < T) issue_load(nxt, stage);
    }
  }
  if (tid == 0) bulk_wait_all();
}

int launch_transpose(const void* in, void* out, int64_t M, int64_t N, const Sched& sched, const int32_t* perm_dev,
                     int32_t* status_dev, cudaStream_t stream) {
  CUtensorMap tmIn, tmOut;
  int rc = make_map(&tmIn, in, M, N, kTrTile, false);
  if (rc != SP_OK) return rc;
  rc = make_map(&tmOut, out, N, M, kTrTile, false);
  if (rc != SP_OK) return rc;
  static uint64_t configured = 0;   // one bit per device
  cudaError_t e;
  if (first_use_on_this_device(configured)) {
    e = cudaFuncSetAttribute(transpose_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTrSmem);
    if (e != cudaSuccess) { configured = 0; set_error("cudaFuncSetAttribute failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
  }
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    set_error("cannot query the device");
    return SP_ERR_CUDA;
  }
  int64_t grid = (int64_t)sms * kTrCtasPerSm;
  if (grid > sched.T) grid = sched.T;
  TransposeArgs args;
  args.perm = perm_dev;
  args.status = status_dev;
  args.sched = sched;
  transpose_kernel<<<(unsigned)grid, kTrThreads, kTrSmem, stream>>>(tmIn, tmOut, args);
  e = cudaGetLastError();
  if (e != cudaSuccess) { set_error("transpose launch failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
  return SP_OK;
}

}  // namespace sp
