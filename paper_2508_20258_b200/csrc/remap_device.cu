// Device evaluation of the tile-order remaps, and the block-dispatch probe.
#include "internal.h"

namespace sp {

constexpr int kBuildThreads = 1024;

// Exclusive block-wide prefix sum of one int per thread; *total receives the block sum.
__device__ int block_exclusive_scan(int v, int* warp_sums, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int w = warp_sums[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += n;
    }
    warp_sums[lane] = w;  // inclusive sums of the warps
  }
  __syncthreads();
  const int before = warp == 0 ? 0 : warp_sums[warp - 1];
  *total = warp_sums[31];
  __syncthreads();
  return before + inc - v;
}

// Curve walk over one sub-grid: cell d is kept when inside the grid; its rank among the
// kept cells is its index in that half.
__device__ void build_curve(const Sched c, int kind, int half, bool split, int rows, int cols, int row0, int col0,
                            int32_t* out, int* warp_sums) {
  const int k = curve_order(rows, cols);
  const uint32_t cells = 1u << (2 * k);
  int base = 0;
  for (uint32_t start = 0; start < cells; start += kBuildThreads) {
    const uint32_t d = start + threadIdx.x;
    int tm = 0, tn = 0;
    const int keep = (d < cells) && curve_cell(kind, k, rows, cols, d, tm, tn);
    int total;
    const int rank = block_exclusive_scan(keep, warp_sums, &total);
    if (keep) {
      const int idx = base + rank;
      const int slot = split ? die_split_slot(c, half, idx) : idx;
      out[slot] = (row0 + tm) * c.Tn + col0 + tn;
    }
    base += total;
  }
}

__global__ void __launch_bounds__(kBuildThreads) build_perm_kernel(const Sched c, int32_t* __restrict__ out) {
  __shared__ int warp_sums[32];
  if (arithmetic_scheme(c)) {
    for (int s = blockIdx.x * kBuildThreads + threadIdx.x; s < c.T; s += gridDim.x * kBuildThreads)
      out[s] = slot_to_tile(c, s);
    return;
  }
  if (blockIdx.x != 0) return;
  if (c.scheme == kMorton || c.scheme == kHilbert) {
    build_curve(c, c.scheme, 0, false, c.Tm, c.Tn, 0, 0, out, warp_sums);
  } else if (c.scheme == kDieSplit) {
    const int cut = c.axis == 0 ? (c.Tm + 1) / 2 : (c.Tn + 1) / 2;
    for (int half = 0; half < 2; ++half) {
      const int rows = c.axis == 0 ? (half ? c.Tm - cut : cut) : c.Tm;
      const int cols = c.axis == 0 ? c.Tn : (half ? c.Tn - cut : cut);
      if (rows == 0 || cols == 0) continue;
      build_curve(c, c.inner, half, true, rows, cols, (c.axis == 0 && half) ? cut : 0,
                  (c.axis == 1 && half) ? cut : 0, out, warp_sums);
    }
  }
}

cudaError_t launch_build_perm(const Sched& c, int32_t* out_dev, cudaStream_t stream) {
  int blocks = 1;
  if (arithmetic_scheme(c)) {
    blocks = (c.T + kBuildThreads - 1) / kBuildThreads;
    if (blocks > 256) blocks = 256;
  }
  build_perm_kernel<<<blocks, kBuildThreads, 0, stream>>>(c, out_dev);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ dispatch probe
__global__ void probe_dispatch_kernel(int32_t* smid, unsigned long long* start) {
  if (threadIdx.x == 0) {
    unsigned s;
    unsigned long long t;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(s));
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    smid[blockIdx.x] = (int32_t)s;
    start[blockIdx.x] = t;
  }
  // stay resident for a moment so later blocks cannot reuse this SM within one wave
  const long long t0 = clock64();
  while (clock64() - t0 < 20000) { }
}

int probe_dispatch(int n_blocks, int cluster, int32_t* smid_host, uint64_t* start_host) {
  int32_t* d_smid = nullptr;
  unsigned long long* d_start = nullptr;
  cudaError_t e = cudaMalloc(&d_smid, sizeof(int32_t) * (size_t)n_blocks);
  if (e == cudaSuccess) e = cudaMalloc(&d_start, sizeof(unsigned long long) * (size_t)n_blocks);
  if (e == cudaSuccess) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_blocks);
    cfg.blockDim = dim3(128);
    // the GEMM kernel is one CTA per SM: ask for enough shared memory that the probe is too
    cfg.dynamicSmemBytes = 200 * 1024;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaFuncSetAttribute(probe_dispatch_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaLaunchKernelEx(&cfg, probe_dispatch_kernel, d_smid, d_start);
  }
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(smid_host, d_smid, sizeof(int32_t) * (size_t)n_blocks, cudaMemcpyDeviceToHost);
  if (e == cudaSuccess) e = cudaMemcpy(start_host, d_start, sizeof(uint64_t) * (size_t)n_blocks, cudaMemcpyDeviceToHost);
  cudaFree(d_smid);
  cudaFree(d_start);
  if (e != cudaSuccess) {
    set_error("dispatch probe failed: %s", cudaGetErrorString(e));
    return SP_ERR_CUDA;
  }
  return SP_OK;
}

}  // namespace sp
