// Topology probe: which SMs sit on which half of the L2 (which die)?
//
// The paper hands its optimiser the number of XCDs and their private L2s as documented
// facts.  For B200 no such table is documented, so it is measured: every SM in turn times
// first-touch loads of the same set of cache lines, each line freshly written before the
// round so that it lives at its home L2 slice only.  A line homed on the SM's own half
// answers faster than one homed on the other half; SMs whose fast/slow patterns agree are
// on the same half.  All loops are bounded; nothing waits on another kernel.
#include <algorithm>
#include <vector>

#include "internal.h"

namespace sp {

constexpr int kProbeLines = SP_PROBE_LINES;
constexpr int kProbeBytes = 4 << 20;
constexpr int kProbeRepeats = 2;

__global__ void probe_reset_kernel(uint32_t* buf, const uint32_t* offsets, int n, uint32_t value) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) buf[offsets[i] / 4] = value + i;
  if (i == 0) buf[kProbeBytes / 4 - 32] = value;   // the line used to warm the TLB
  __threadfence();
}

// One CTA per SM (the shared-memory request makes them exclusive); only the CTA that finds
// itself on `target` measures.  lat[i] = min over repeats of the load latency of line i in cycles.
__global__ void probe_measure_kernel(const uint32_t* buf, const uint32_t* offsets, int n, int target, uint32_t* lat,
                                     uint32_t* sink_out, unsigned long long zero) {
  uint32_t smid;
  asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
  if ((int)smid != target || threadIdx.x != 0) return;
  uint32_t sink = 0, v;
  const uint32_t* warm = buf + (kProbeBytes / 4 - 32);
  asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(v) : "l"(warm) : "memory");
  sink += v;
#pragma unroll 1
  for (int i = 0; i < n; ++i) {
    unsigned long long t0, t1;
    asm volatile("mov.u64 %0, %%clock64;" : "=l"(t0) :: "memory");
    // the address depends on the first clock value (`zero` is 0 at run time, unknown to the compiler), so the load
    // cannot be issued early; the add consumes the loaded value before the second clock read
    const uint32_t* p = buf + offsets[i] / 4 + (t0 & zero);
    asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    asm volatile("add.u32 %0, %0, %1;" : "+r"(sink) : "r"(v) : "memory");
    asm volatile("mov.u64 %0, %%clock64;" : "=l"(t1) : "r"(sink) : "memory");
    const uint32_t d = (uint32_t)(t1 - t0);
    if (lat[i] == 0 || d < lat[i]) lat[i] = d;
  }
  *sink_out = sink;
}

int probe_topology(int32_t* sm_to_die_host, int32_t* n_sm_out, float* confidence, uint32_t* lat_host) {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess || sms <= 0 || sms > 1024) { set_error("cannot query the device"); return SP_ERR_CUDA; }

  // pseudo-random, distinct, 128-byte-aligned line offsets inside one 4 MiB buffer
  std::vector<uint32_t> offs(kProbeLines);
  uint32_t x = 12345u;
  std::vector<uint8_t> used(kProbeBytes / 128, 0);
  for (int i = 0; i < kProbeLines; ++i) {
    uint32_t line;
    do { x = x * 1664525u + 1013904223u; line = (x >> 8) % (kProbeBytes / 128 - 64); } while (used[line]);
    used[line] = 1;
    offs[i] = line * 128u;
  }
  uint32_t *d_buf = nullptr, *d_offs = nullptr, *d_lat = nullptr, *d_sink = nullptr;
  e = cudaMalloc(&d_buf, kProbeBytes);
  if (e == cudaSuccess) e = cudaMalloc(&d_offs, sizeof(uint32_t) * kProbeLines);
  if (e == cudaSuccess) e = cudaMalloc(&d_lat, sizeof(uint32_t) * (size_t)sms * kProbeLines);
  if (e == cudaSuccess) e = cudaMalloc(&d_sink, sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMemset(d_buf, 0, kProbeBytes);
  if (e == cudaSuccess) e = cudaMemset(d_lat, 0, sizeof(uint32_t) * (size_t)sms * kProbeLines);
  if (e == cudaSuccess) e = cudaMemcpy(d_offs, offs.data(), sizeof(uint32_t) * kProbeLines, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(probe_measure_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  for (int rep = 0; rep < kProbeRepeats && e == cudaSuccess; ++rep) {
    for (int t = 0; t < sms && e == cudaSuccess; ++t) {
      probe_reset_kernel<<<(kProbeLines + 127) / 128, 128>>>(d_buf, d_offs, kProbeLines, (uint32_t)(rep * 4096 + t));
      probe_measure_kernel<<<sms, 32, 200 * 1024>>>(d_buf, d_offs, kProbeLines, t, d_lat + (size_t)t * kProbeLines, d_sink, 0ull);
      e = cudaGetLastError();
    }
  }
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  std::vector<uint32_t> lat((size_t)sms * kProbeLines, 0);
  if (e == cudaSuccess) e = cudaMemcpy(lat.data(), d_lat, sizeof(uint32_t) * lat.size(), cudaMemcpyDeviceToHost);
  cudaFree(d_buf); cudaFree(d_offs); cudaFree(d_lat); cudaFree(d_sink);
  if (e != cudaSuccess) { set_error("topology probe failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
  if (lat_host) std::copy(lat.begin(), lat.end(), lat_host);

  // sign pattern of each SM against the per-line median; SMs are grouped by agreement with a reference SM
  std::vector<float> med(kProbeLines);
  std::vector<uint32_t> col(sms);
  for (int i = 0; i < kProbeLines; ++i) {
    int n = 0;
    for (int t = 0; t < sms; ++t) if (lat[(size_t)t * kProbeLines + i]) col[n++] = lat[(size_t)t * kProbeLines + i];
    if (n == 0) { med[i] = 0; continue; }
    std::sort(col.begin(), col.begin() + n);
    med[i] = 0.5f * (col[(n - 1) / 2] + col[n / 2]);
  }
  int ref = -1;
  for (int t = 0; t < sms && ref < 0; ++t) if (lat[(size_t)t * kProbeLines]) ref = t;
  double conf_sum = 0;
  int measured = 0;
  for (int t = 0; t < sms; ++t) {
    sm_to_die_host[t] = -1;
    if (ref < 0 || !lat[(size_t)t * kProbeLines]) continue;
    int agree = 0, total = 0;
    for (int i = 0; i < kProbeLines; ++i) {
      const float a = (float)lat[(size_t)ref * kProbeLines + i] - med[i], b = (float)lat[(size_t)t * kProbeLines + i] - med[i];
      if (a == 0 || b == 0) continue;
      if (lat[(size_t)ref * kProbeLines + i] < 64 || lat[(size_t)t * kProbeLines + i] < 64) continue;  // not a memory access
      agree += (a > 0) == (b > 0);
      ++total;
    }
    if (total == 0) continue;
    const double c = 2.0 * agree / total - 1.0;     // +1: same pattern as the reference, -1: complementary
    sm_to_die_host[t] = c >= 0 ? 0 : 1;
    conf_sum += c >= 0 ? c : -c;
    ++measured;
  }
  *n_sm_out = sms;
  *confidence = measured ? (float)(conf_sum / measured) : 0.f;
  return SP_OK;
}

}  // namespace sp

namespace sp {

// ------------------------------------------------------------------ effective L2 capacity
// Every participating CTA (one per SM) reads the whole working set with 16-byte loads that bypass L1; the pass is
// repeated, so the rate of the later passes tells whether the set still fits in what the L2 can hold for these readers.
// With `half` >= 0 only the CTAs on that L2 half take part.
__global__ void probe_capacity_kernel(const uint4* __restrict__ buf, size_t n16, int passes, int half, const uint32_t* die_mask,
                                      uint32_t* sink_out) {
  uint32_t smid;
  asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
  if (half >= 0 && (int)((die_mask[(smid >> 5) & 7] >> (smid & 31)) & 1u) != half) return;
  uint32_t acc = 0;
  for (int p = 0; p < passes; ++p) {
    // CTAs start at different offsets so that they do not all hit the same lines at the same time
    const size_t start = ((size_t)blockIdx.x * 4099u * 64u) % n16;
    for (size_t i = threadIdx.x; i < n16; i += blockDim.x) {
      size_t j = start + i;
      if (j >= n16) j -= n16;
      uint4 v;
      asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(buf + j));
      acc += v.x ^ v.y ^ v.z ^ v.w;
    }
  }
  if (acc == 0x12345678u) *sink_out = acc;   // keeps the loads alive
}

int probe_l2_capacity(int n_sizes, const int64_t* sizes_bytes, int half, const uint32_t* die_mask_host, float* gbps_out) {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    set_error("cannot query the device");
    return SP_ERR_CUDA;
  }
  int64_t max_bytes = 0;
  for (int i = 0; i < n_sizes; ++i) {
    if (sizes_bytes[i] < 4096 || sizes_bytes[i] > (1ll << 30) || (sizes_bytes[i] % 16) != 0) { set_error("bad working-set size"); return SP_ERR_INVALID_ARG; }
    if (sizes_bytes[i] > max_bytes) max_bytes = sizes_bytes[i];
  }
  uint4* d_buf = nullptr;
  uint32_t *d_mask = nullptr, *d_sink = nullptr;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  cudaError_t e = cudaMalloc(&d_buf, (size_t)max_bytes);
  if (e == cudaSuccess) e = cudaMalloc(&d_mask, 8 * sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMalloc(&d_sink, sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMemset(d_buf, 1, (size_t)max_bytes);
  if (e == cudaSuccess) e = cudaMemcpy(d_mask, die_mask_host, 8 * sizeof(uint32_t), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(probe_capacity_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  const int passes = 4;
  for (int i = 0; i < n_sizes && e == cudaSuccess; ++i) {
    const size_t n16 = (size_t)sizes_bytes[i] / 16;
    probe_capacity_kernel<<<sms, 512, 200 * 1024>>>(d_buf, n16, 1, half, d_mask, d_sink);          // warm pass
    cudaEventRecord(e0);
    probe_capacity_kernel<<<sms, 512, 200 * 1024>>>(d_buf, n16, passes, half, d_mask, d_sink);
    cudaEventRecord(e1);
    e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    int readers = sms;
    if (half >= 0) {
      readers = 0;
      for (int s = 0; s < sms; ++s) readers += (int)((die_mask_host[(s >> 5) & 7] >> (s & 31)) & 1u) == half;
    }
    gbps_out[i] = ms > 0.f ? (float)((double)sizes_bytes[i] * passes * readers / (ms * 1e6)) : 0.f;
  }
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  cudaFree(d_buf); cudaFree(d_mask); cudaFree(d_sink);
  if (e != cudaSuccess) { set_error("capacity probe failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
  return SP_OK;
}

}  // namespace sp
