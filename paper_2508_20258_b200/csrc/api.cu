// C ABI of libswizzleperf.so: argument validation, the host remap, caches, status.
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <deque>
#include <mutex>
#include <vector>

#include "internal.h"
#include "streamk.cuh"

namespace sp {

static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof g_err, fmt, ap);
  va_end(ap);
}

static bool plain_inner(int s) { return s >= kRow && s <= kHilbert; }

int resolve_sched(int64_t M, int64_t N, int32_t tileM, int32_t tileN, int scheme, const sp_params* p, Sched* out) {
  if (M <= 0 || N <= 0 || tileM <= 0 || tileN <= 0) {
    set_error("sizes must be positive (M=%lld N=%lld tileM=%d tileN=%d)", (long long)M, (long long)N, tileM, tileN);
    return SP_ERR_INVALID_ARG;
  }
  if (p && p->struct_size != sizeof(sp_params)) {
    set_error("sp_params.struct_size is %u, expected %zu", p->struct_size, sizeof(sp_params));
    return SP_ERR_INVALID_ARG;
  }
  const int64_t Tm = (M + tileM - 1) / tileM, Tn = (N + tileN - 1) / tileN;
  if (Tm > kMaxTiles || Tn > kMaxTiles || Tm * Tn > kMaxTiles) {
    set_error("too many tiles (%lld x %lld)", (long long)Tm, (long long)Tn);
    return SP_ERR_INVALID_ARG;
  }
  Sched c;
  memset(&c, 0, sizeof c);
  c.scheme = scheme;
  c.Tm = (int)Tm; c.Tn = (int)Tn; c.T = (int)(Tm * Tn);
  c.group = 1; c.X = 1; c.W = c.T; c.inner_group = 1;
  switch (scheme) {
    case kRow: case kCol: case kMorton: case kHilbert: case kHilbertRect: break;
    case kGroupM: case kGroupN:
      if (!p || p->group < 1) { set_error("group must be >= 1"); return SP_ERR_INVALID_ARG; }
      c.group = p->group;
      c.serp = (p->flags & SP_FLAG_SERPENTINE) != 0;
      break;
    case kXcd:
      if (!p || p->num_xcds < 1) { set_error("num_xcds must be >= 1"); return SP_ERR_INVALID_ARG; }
      if (p->wave < 0) { set_error("wave must be >= 0"); return SP_ERR_INVALID_ARG; }
      c.X = p->num_xcds;
      c.W = (p->wave == 0 || p->wave > c.T) ? c.T : p->wave;
      c.balanced = p->xcd_balanced != 0;
      break;
    case kDieSplit:
      if (!p) { set_error("SP_DIE_SPLIT needs parameters"); return SP_ERR_INVALID_ARG; }
      if (p->split_axis != 0 && p->split_axis != 1) { set_error("split_axis must be 0 or 1"); return SP_ERR_INVALID_ARG; }
      if (!plain_inner(p->inner_scheme)) { set_error("inner_scheme must be a plain order"); return SP_ERR_INVALID_ARG; }
      c.axis = p->split_axis; c.inner = p->inner_scheme; c.interleave = p->interleave != 0;
      if (c.inner == kGroupM || c.inner == kGroupN) {
        if (p->inner_group < 1) { set_error("inner_group must be >= 1"); return SP_ERR_INVALID_ARG; }
        c.inner_group = p->inner_group;
        c.serp = (p->flags & SP_FLAG_SERPENTINE) != 0;
      }
      break;
    case kCustom:
      if (!p || !p->custom_perm) { set_error("SP_CUSTOM needs custom_perm"); return SP_ERR_INVALID_ARG; }
      break;
    default:
      set_error("unknown scheme %d", scheme);
      return SP_ERR_INVALID_ARG;
  }
  if (scheme == kHilbertRect && ((int64_t)c.Tm > 32768 || (int64_t)c.Tn > 32768)) {
    set_error("SP_HILBERT_RECT supports grids up to 32768 tiles per side");
    return SP_ERR_UNSUPPORTED;
  }
  const bool curve = scheme == kMorton || scheme == kHilbert ||
                     (scheme == kDieSplit && (c.inner == kMorton || c.inner == kHilbert));
  if (curve && (c.Tm > kMaxCurveSide || c.Tn > kMaxCurveSide)) {
    set_error("curve orders support grids up to %d tiles per side", kMaxCurveSide);
    return SP_ERR_UNSUPPORTED;
  }
  // The generalised Hilbert curve is arithmetic (no rank among skipped cells is needed) but costs a few hundred
  // instructions per cell: kernels read it from a table, which the device builder fills with the same function.
  c.use_table = (arithmetic_scheme(c) && scheme != kHilbertRect) ? 0 : 1;
  *out = c;
  return SP_OK;
}

static bool bijective(const std::vector<int32_t>& perm, int T) {
  if ((int)perm.size() != T) return false;
  std::vector<uint8_t> seen((size_t)T, 0);
  for (int32_t t : perm) {
    if (t < 0 || t >= T || seen[(size_t)t]) return false;
    seen[(size_t)t] = 1;
  }
  return true;
}

// Walks a curve over a (rows x cols) sub-grid and emits grid ids of the whole grid.
template <typename Emit>
static void walk_curve(int kind, int rows, int cols, int row0, int col0, int Tn, Emit emit) {
  const int k = curve_order(rows, cols);
  const uint64_t cells = 1ull << (2 * k);
  int idx = 0;
  for (uint64_t d = 0; d < cells; ++d) {
    int tm, tn;
    if (curve_cell(kind, k, rows, cols, (uint32_t)d, tm, tn)) emit(idx++, (row0 + tm) * Tn + col0 + tn);
  }
}

int build_perm_host(const Sched& c, const int32_t* custom, std::vector<int32_t>& perm) {
  perm.assign((size_t)c.T, -1);
  if (c.scheme == kCustom) {
    if (!custom) { set_error("SP_CUSTOM needs custom_perm"); return SP_ERR_INVALID_ARG; }
    for (int s = 0; s < c.T; ++s) perm[(size_t)s] = custom[s];
  } else if (arithmetic_scheme(c)) {
    for (int s = 0; s < c.T; ++s) perm[(size_t)s] = slot_to_tile(c, s);
  } else if (c.scheme == kMorton || c.scheme == kHilbert) {
    walk_curve(c.scheme, c.Tm, c.Tn, 0, 0, c.Tn, [&](int idx, int t) { perm[(size_t)idx] = t; });
  } else {  // DIE_SPLIT with a curve inside each half
    for (int half = 0; half < 2; ++half) {
      const int cut = c.axis == 0 ? (c.Tm + 1) / 2 : (c.Tn + 1) / 2;
      const int rows = c.axis == 0 ? (half ? c.Tm - cut : cut) : c.Tm;
      const int cols = c.axis == 0 ? c.Tn : (half ? c.Tn - cut : cut);
      if (rows == 0 || cols == 0) continue;
      walk_curve(c.inner, rows, cols, (c.axis == 0 && half) ? cut : 0, (c.axis == 1 && half) ? cut : 0, c.Tn,
                 [&](int idx, int t) { perm[(size_t)die_split_slot(c, half, idx)] = t; });
    }
  }
  if (!bijective(perm, c.T)) {
    set_error("remap (scheme %d) is not a bijection on [0,%d)", c.scheme, c.T);
    return SP_ERR_NOT_BIJECTIVE;
  }
  return SP_OK;
}

// ------------------------------------------------------------------ per-device caches
struct TableEntry {
  Sched key;
  uint64_t custom_hash;
  int32_t* dev;
  uint64_t stamp;
};

constexpr int kHostChunks = 32;  // sp_gemm_host splits M into at most this many row blocks

struct DeviceState {
  int device = -1;
  int32_t* status = nullptr;
  std::vector<TableEntry> tables;
  unsigned die_pair_next = 0;   // rotation over the counter pairs
  int die_known = 0;            // 0: not probed, 1: usable map, -1: probe found no two-way structure
  int sms_on_die[2] = {0, 0};
  uint32_t die_mask[8] = {};
  void* softmax_ws = nullptr;   // partial maxima and sums of the two-phase softmax (grow-only)
  size_t softmax_ws_bytes = 0;
  void* staging = nullptr;      // device copies of A, B, C for sp_gemm_host (grow-only)
  size_t staging_bytes = 0;
  cudaStream_t copy_in = nullptr, copy_out = nullptr;   // sp_gemm_host: copies overlap the chunked compute
  // SP_FLAG_STREAM_K: one workspace (partial tiles + flags) per stream that has asked for it, so that launches on
  // different streams never share one; launches on one stream are ordered by the stream
  struct SkSpace { cudaStream_t stream; void* mem; int32_t epoch; };
  std::vector<SkSpace> sk_spaces;
  cudaEvent_t ev[2 * kHostChunks + 3] = {};
};

static std::mutex g_mu;
static std::deque<DeviceState> g_devs;   // a deque: entries keep their address when another device is added
static uint64_t g_stamp = 0;
constexpr size_t kMaxTables = 64;

constexpr size_t kMaxSkStreams = 8;
constexpr int kDiePairs = 64;   // die-pinned launches that may be in flight at once on one device (different streams)
constexpr int kDieWords = 5;    // counters per die-pinned launch: arrivals per half (2), units finished, queue heads (2)
static std::mutex g_valid_mu;
static std::vector<Sched> g_validated;

bool already_validated(const Sched& c) {
  std::lock_guard<std::mutex> lock(g_valid_mu);
  for (const Sched& v : g_validated) if (memcmp(&v, &c, sizeof c) == 0) return true;
  return false;
}

void remember_validated(const Sched& c) {
  std::lock_guard<std::mutex> lock(g_valid_mu);
  if (g_validated.size() >= 256) g_validated.erase(g_validated.begin());
  g_validated.push_back(c);
}

static DeviceState* device_state(int dev) {
  for (auto& d : g_devs) if (d.device == dev) return &d;
  g_devs.emplace_back();
  g_devs.back().device = dev;
  return &g_devs.back();
}

static uint64_t fnv(const int32_t* v, int n) {
  uint64_t h = 1469598103934665603ull;
  for (int i = 0; i < n; ++i) { h ^= (uint32_t)v[i]; h *= 1099511628211ull; }
  return h;
}

#define SP_CUDA(call)                                                             \
  do {                                                                            \
    cudaError_t e_ = (call);                                                      \
    if (e_ != cudaSuccess) {                                                      \
      set_error("%s failed: %s", #call, cudaGetErrorString(e_));                  \
      return SP_ERR_CUDA;                                                         \
    }                                                                             \
  } while (0)

int current_device(int* dev) {
  // the checks below are per (host thread, device): once passed, a call costs one cudaGetDevice
  static thread_local int checked_dev = -1;
  if (checked_dev >= 0) {
    int d = -1;
    if (cudaGetDevice(&d) == cudaSuccess && d == checked_dev) { *dev = d; return SP_OK; }
    checked_dev = -1;
  }
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess || n == 0) {
    cudaGetLastError();
    set_error("no CUDA device");
    return SP_ERR_DEVICE;
  }
  SP_CUDA(cudaGetDevice(dev));
  // A host thread that has made no runtime call yet has no context bound, and the tensor maps are encoded through the
  // driver API, which needs one: selecting the device it already has binds the primary context to this thread.
  SP_CUDA(cudaSetDevice(*dev));
  int major = 0;
  SP_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, *dev));
  if (major != 10) {
    set_error("device %d has compute capability %d.x; this library is sm_100a only", *dev, major);
    return SP_ERR_DEVICE;
  }
  checked_dev = *dev;
  return SP_OK;
}

static int get_status_word(DeviceState* ds) {
  if (!ds->status) {
    // status word, then kDiePairs counter sets (arrivals on half 0, arrivals on half 1, units finished, next ticket of
    // half 0, of half 1) handed to die-pinned launches in rotation; the last unit of a launch to finish puts its set
    // back to zero
    SP_CUDA(cudaMalloc(&ds->status, (2 + kDieWords * kDiePairs) * sizeof(int32_t)));
    SP_CUDA(cudaMemset(ds->status, 0, (2 + kDieWords * kDiePairs) * sizeof(int32_t)));
  }
  return SP_OK;
}

// SM -> L2-half map of the device, probed once.  Usable only if the probe is confident, the halves
// are equal and the two SMs of every CTA pair share a half.
static int get_die_map(DeviceState* ds) {
  if (ds->die_known == 0) {
    std::vector<int32_t> die(1024, -1);
    int n = 0;
    float conf = 0.f;
    int rc = probe_topology(die.data(), &n, &conf, nullptr);
    if (rc != SP_OK) return rc;
    bool ok = conf >= 0.8f && n <= 256;
    int cnt[2] = {0, 0};
    for (int i = 0; i < n && ok; ++i) {
      if (die[i] < 0) { ok = false; break; }
      cnt[die[i]]++;
      if (die[i]) ds->die_mask[i >> 5] |= 1u << (i & 31);
      if ((i & 1) && die[i] != die[i - 1]) ok = false;
    }
    ok = ok && cnt[0] > 0 && cnt[1] > 0 && (cnt[0] % 2) == 0 && (cnt[1] % 2) == 0;
    ds->sms_on_die[0] = cnt[0]; ds->sms_on_die[1] = cnt[1];
    ds->die_known = ok ? 1 : -1;
  }
  if (ds->die_known < 0) { set_error("the topology probe found no usable two-way L2 structure on this device"); return SP_ERR_UNSUPPORTED; }
  return SP_OK;
}

// Device table for a table scheme; built by the device builder (or copied for SP_CUSTOM).  The build runs once per
// table and is complete when this returns: an entry is published in the cache only after the stream that filled it
// has been synchronised, so a later call on any stream or host thread that finds it may launch at once.
static int get_table(DeviceState* ds, const Sched& c, const std::vector<int32_t>& host_perm, bool is_custom,
                     cudaStream_t stream, const int32_t** out) {
  const uint64_t h = is_custom ? fnv(host_perm.data(), c.T) : 0;
  for (auto& e : ds->tables)
    if (memcmp(&e.key, &c, sizeof c) == 0 && e.custom_hash == h) { e.stamp = ++g_stamp; *out = e.dev; return SP_OK; }
  if (ds->tables.size() >= kMaxTables) {
    size_t lru = 0;
    for (size_t i = 1; i < ds->tables.size(); ++i) if (ds->tables[i].stamp < ds->tables[lru].stamp) lru = i;
    cudaFree(ds->tables[lru].dev);  // synchronises: no kernel can still be reading it afterwards
    ds->tables.erase(ds->tables.begin() + (long)lru);
  }
  TableEntry e;
  e.key = c; e.custom_hash = h; e.stamp = ++g_stamp; e.dev = nullptr;
  SP_CUDA(cudaMalloc(&e.dev, sizeof(int32_t) * (size_t)c.T));
  cudaError_t ce;
  if (is_custom)   // pageable source: the copy has been staged when the call returns, so host_perm may die
    ce = cudaMemcpyAsync(e.dev, host_perm.data(), sizeof(int32_t) * (size_t)c.T, cudaMemcpyHostToDevice, stream);
  else
    ce = launch_build_perm(c, e.dev, stream);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(stream);
  if (ce != cudaSuccess) { cudaFree(e.dev); set_error("filling the tile table failed: %s", cudaGetErrorString(ce)); return SP_ERR_CUDA; }
  ds->tables.push_back(e);
  *out = e.dev;
  return SP_OK;
}

// Argument checks shared by every GEMM entry point; fills the resolved shape options.
int validate_gemm_args(const void* A, const void* B, const void* C, int64_t M, int64_t N, int64_t K, const sp_params* params,
                       int* tile_m_out, int* tile_n_out, int* out_f32_out, int* b_nk_out) {
  if (!A || !B || !C) { set_error("A, B and C must not be NULL"); return SP_ERR_INVALID_ARG; }
  if (M <= 0 || N <= 0 || K <= 0) { set_error("M, N, K must be positive"); return SP_ERR_INVALID_ARG; }
  if (M >= (1ll << 31) || N >= (1ll << 31) || K >= (1ll << 31)) { set_error("dimension too large"); return SP_ERR_UNSUPPORTED; }
  if (params && params->struct_size != sizeof(sp_params)) {
    set_error("sp_params.struct_size is %u, expected %zu", params->struct_size, sizeof(sp_params));
    return SP_ERR_INVALID_ARG;
  }
  int tile_m = params ? params->tile_m : 0, tile_n = params ? params->tile_n : 0;
  if (tile_m == 0 && tile_n == 0) { tile_m = 256; tile_n = 256; }
  if (!(((tile_m == 128 || tile_m == 256) && (tile_n == 128 || tile_n == 256)) || (tile_m == 256 && tile_n == 512))) {
    set_error("unsupported tile %dx%d (supported: 128x128, 128x256, 256x128, 256x256, 256x512)", tile_m, tile_n);
    return SP_ERR_UNSUPPORTED;
  }
  const int out_f32 = params ? params->out_dtype : 0;
  const int b_nk = params ? params->b_layout : 0;
  if ((out_f32 != 0 && out_f32 != 1) || (b_nk != 0 && b_nk != 1)) { set_error("bad out_dtype / b_layout"); return SP_ERR_INVALID_ARG; }
  if (((uintptr_t)A | (uintptr_t)B | (uintptr_t)C) & 15u) { set_error("A, B, C must be 16-byte aligned"); return SP_ERR_ALIGNMENT; }
  if ((K % 8) != 0 || (N % 8) != 0) { set_error("K and N must be multiples of 8 (16-byte row pitch)"); return SP_ERR_ALIGNMENT; }
  *tile_m_out = tile_m; *tile_n_out = tile_n; *out_f32_out = out_f32; *b_nk_out = b_nk;
  return SP_OK;
}

// The flags that change only how memory is walked or cached (no scratch memory, no scheduling state): K direction per
// round and L2 eviction priorities.  Shared by every GEMM entry point.
int apply_memory_flags(const sp_params* params, GemmCall* call) {
  call->k_alternate = 0; call->hint_a = call->hint_b = call->hint_c = 0;
  if (!params) return SP_OK;
  const uint32_t f = params->flags;
  if (((f & SP_FLAG_HINT_A_EVICT_FIRST) && (f & SP_FLAG_HINT_A_EVICT_LAST)) ||
      ((f & SP_FLAG_HINT_B_EVICT_FIRST) && (f & SP_FLAG_HINT_B_EVICT_LAST))) {
    set_error("an operand cannot be both evict_first and evict_last");
    return SP_ERR_INVALID_ARG;
  }
  call->k_alternate = (f & SP_FLAG_K_ALTERNATE) ? 1 : 0;
  call->hint_a = (f & SP_FLAG_HINT_A_EVICT_FIRST) ? 1 : (f & SP_FLAG_HINT_A_EVICT_LAST) ? 2 : 0;
  call->hint_b = (f & SP_FLAG_HINT_B_EVICT_FIRST) ? 1 : (f & SP_FLAG_HINT_B_EVICT_LAST) ? 2 : 0;
  call->hint_c = (f & SP_FLAG_HINT_C_EVICT_FIRST) ? 1 : 0;
  return SP_OK;
}

static int gemm_common(const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t K, int scheme,
                       const sp_params* params, void* stream, sp_trace_rec* trace, bool want_trace) {
  if (want_trace && !trace) { set_error("trace buffer must not be NULL"); return SP_ERR_INVALID_ARG; }
  int tile_m, tile_n, out_f32, b_nk;
  int rc0 = validate_gemm_args(A, B, C, M, N, K, params, &tile_m, &tile_n, &out_f32, &b_nk);
  if (rc0 != SP_OK) return rc0;

  GemmCall call;
  memset(&call, 0, sizeof call);
  int rc = resolve_sched(M, N, tile_m, tile_n, scheme, params, &call.sched);
  if (rc != SP_OK) return rc;
  // Bijectivity gate.  A (grid, scheme, parameters) that passed once is remembered, so the hot
  // path does no O(T) host work; caller tables are re-checked on every call (their contents may change).
  std::vector<int32_t> host_perm;
  if (scheme == kCustom || !already_validated(call.sched)) {
    rc = build_perm_host(call.sched, params ? params->custom_perm : nullptr, host_perm);
    if (rc != SP_OK) return rc;
    if (scheme != kCustom) remember_validated(call.sched);
  }

  int dev = 0;
  rc = current_device(&dev);
  if (rc != SP_OK) return rc;
  std::lock_guard<std::mutex> lock(g_mu);
  DeviceState* ds = device_state(dev);
  rc = get_status_word(ds);
  if (rc != SP_OK) return rc;
  call.A = A; call.B = B; call.C = C; call.M = M; call.N = N; call.K = K;
  call.tile_m = tile_m; call.tile_n = tile_n; call.out_f32 = out_f32; call.b_nk = b_nk;
  call.status_dev = ds->status;
  call.trace_dev = want_trace ? trace : nullptr;
  call.stream = (cudaStream_t)stream;
  call.perm_dev = nullptr;
  if (call.sched.use_table) {
    rc = get_table(ds, call.sched, host_perm, scheme == kCustom, call.stream, &call.perm_dev);
    if (rc != SP_OK) return rc;
  }
  rc = apply_memory_flags(params, &call);
  if (rc != SP_OK) return rc;
  if (params && (params->flags & SP_FLAG_OVERLAP)) {
    if (want_trace || (params->flags & (SP_FLAG_DIE_PINNED | SP_FLAG_STREAM_K))) {
      set_error("SP_FLAG_OVERLAP cannot be combined with tracing, SP_FLAG_DIE_PINNED or SP_FLAG_STREAM_K");
      return SP_ERR_INVALID_ARG;
    }
    call.overlap = 1;
  }
  if (params && (params->flags & SP_FLAG_STEAL) && !(params->flags & SP_FLAG_DIE_PINNED)) {
    set_error("SP_FLAG_STEAL is a mode of SP_FLAG_DIE_PINNED (per-half queues)");
    return SP_ERR_INVALID_ARG;
  }
  if (params && (params->flags & SP_FLAG_DIE_PINNED)) {
    if (scheme != kDieSplit || call.sched.interleave) {
      set_error("SP_FLAG_DIE_PINNED needs SP_DIE_SPLIT with interleave = 0");
      return SP_ERR_INVALID_ARG;
    }
    rc = get_die_map(ds);
    if (rc != SP_OK) return rc;
    call.pinned = 1;
    call.die_count_dev = ds->status + 2 + kDieWords * (int)(ds->die_pair_next++ % kDiePairs);
    call.steal = (params->flags & SP_FLAG_STEAL) ? 1 : 0;
    call.half0 = die_split_half0(call.sched);
    call.sms_on_die[0] = ds->sms_on_die[0]; call.sms_on_die[1] = ds->sms_on_die[1];
    for (int i = 0; i < 8; ++i) call.die_mask[i] = ds->die_mask[i];
  }
  if (params && (params->flags & SP_FLAG_CLC)) {
    if (params->flags & (SP_FLAG_DIE_PINNED | SP_FLAG_STREAM_K)) {
      set_error("SP_FLAG_CLC cannot be combined with SP_FLAG_DIE_PINNED or SP_FLAG_STREAM_K");
      return SP_ERR_INVALID_ARG;
    }
    call.clc = 1;
  }
  if (params && (params->flags & SP_FLAG_STREAM_K)) {
    if (call.pinned) {
      set_error("SP_FLAG_STREAM_K cannot be combined with SP_FLAG_DIE_PINNED");
      return SP_ERR_INVALID_ARG;
    }
    if (tile_n > 256) { set_error("SP_FLAG_STREAM_K is not implemented for the 256x512 tile"); return SP_ERR_UNSUPPORTED; }
    DeviceState::SkSpace* space = nullptr;
    for (auto& sk : ds->sk_spaces) if (sk.stream == call.stream) space = &sk;
    if (!space) {
      void* mem = nullptr;
      if (ds->sk_spaces.size() >= kMaxSkStreams) {
        set_error("SP_FLAG_STREAM_K is in use on %zu streams already (sp_shutdown releases them)", ds->sk_spaces.size());
        return SP_ERR_UNSUPPORTED;
      }
      SP_CUDA(cudaMalloc(&mem, kSkFlagBytes + kSkWorkspaceBytes));
      cudaError_t ce = cudaMemset(mem, 0, kSkFlagBytes);
      if (ce != cudaSuccess) { cudaFree(mem); set_error("clearing the stream-K flags failed: %s", cudaGetErrorString(ce)); return SP_ERR_CUDA; }
      ds->sk_spaces.push_back({call.stream, mem, 0});
      space = &ds->sk_spaces.back();
    }
    if (space->epoch == INT32_MAX) {   // the flags have seen every value: start over
      SP_CUDA(cudaStreamSynchronize(call.stream));
      SP_CUDA(cudaMemset(space->mem, 0, kSkFlagBytes));
      space->epoch = 0;
    }
    call.stream_k = 1;
    call.sk_epoch = ++space->epoch;
    call.sk_flags_dev = (int32_t*)space->mem;
    call.sk_ws_dev = (float*)((char*)space->mem + kSkFlagBytes);
  }
  return launch_gemm(call);
}

}  // namespace sp

using namespace sp;

extern "C" {

int64_t sp_tile_count(int64_t M, int64_t N, int32_t tileM, int32_t tileN) {
  if (M <= 0 || N <= 0 || tileM <= 0 || tileN <= 0) return -1;
  return ((M + tileM - 1) / tileM) * ((N + tileN - 1) / tileN);
}

int sp_tile_map(int64_t M, int64_t N, int32_t tileM, int32_t tileN, int scheme, const sp_params* params,
                int32_t* out_perm) {
  if (!out_perm) { set_error("out_perm must not be NULL"); return SP_ERR_INVALID_ARG; }
  Sched c;
  int rc = resolve_sched(M, N, tileM, tileN, scheme, params, &c);
  if (rc != SP_OK) return rc;
  std::vector<int32_t> perm;
  rc = build_perm_host(c, params ? params->custom_perm : nullptr, perm);
  if (rc != SP_OK) return rc;
  memcpy(out_perm, perm.data(), sizeof(int32_t) * perm.size());
  return SP_OK;
}

int sp_tile_map_device(int64_t M, int64_t N, int32_t tileM, int32_t tileN, int scheme, const sp_params* params,
                       int32_t* out_perm_dev, void* stream) {
  if (!out_perm_dev) { set_error("out_perm_dev must not be NULL"); return SP_ERR_INVALID_ARG; }
  Sched c;
  int rc = resolve_sched(M, N, tileM, tileN, scheme, params, &c);
  if (rc != SP_OK) return rc;
  std::vector<int32_t> perm;
  rc = build_perm_host(c, params ? params->custom_perm : nullptr, perm);
  if (rc != SP_OK) return rc;
  int dev = 0;
  rc = current_device(&dev);
  if (rc != SP_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  if (scheme == kCustom) {
    SP_CUDA(cudaMemcpyAsync(out_perm_dev, perm.data(), sizeof(int32_t) * perm.size(), cudaMemcpyHostToDevice, st));
    SP_CUDA(cudaStreamSynchronize(st));
    return SP_OK;
  }
  SP_CUDA(launch_build_perm(c, out_perm_dev, st));
  return SP_OK;
}

int sp_streamk_plan(int64_t T, int32_t units, int32_t kblocks, int32_t* first_slot, int32_t* out_segments) {
  if (T <= 0 || T > kMaxTiles || units <= 0 || units > 4096 || kblocks <= 0 || !first_slot || !out_segments) {
    set_error("sp_streamk_plan: bad argument (T=%lld units=%d kblocks=%d)", (long long)T, units, kblocks);
    return SP_ERR_INVALID_ARG;
  }
  const SkPlan p = sk_plan(T, units, kblocks);
  *first_slot = p.first_slot;
  for (int64_t i = 0; i < (int64_t)units * SP_STREAMK_MAX_SEGMENTS * 4; ++i) out_segments[i] = i % 4 == 0 ? -1 : 0;
  for (int u = 0; u < units; ++u) {
    const int n = sk_segments(p, u, kblocks);
    if (n > SP_STREAMK_MAX_SEGMENTS) { set_error("unit %d has %d segments", u, n); return SP_ERR_UNSUPPORTED; }
    for (int j = 0; j < n; ++j) {
      const Work w = sk_segment(p, u, j, kblocks);
      int32_t* o = out_segments + ((size_t)u * SP_STREAMK_MAX_SEGMENTS + j) * 4;
      o[0] = w.slot; o[1] = w.k0; o[2] = w.k1; o[3] = w.kind;
    }
  }
  return SP_OK;
}

int sp_gemm(const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t K, int scheme,
            const sp_params* params, void* stream) {
  return gemm_common(A, B, C, M, N, K, scheme, params, stream, nullptr, false);
}

int sp_gemm_trace(const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t K, int scheme,
                  const sp_params* params, void* stream, sp_trace_rec* trace_dev) {
  return gemm_common(A, B, C, M, N, K, scheme, params, stream, trace_dev, true);
}

int sp_gemm_host(const void* A_host, const void* B_host, void* C_host, int64_t M, int64_t N, int64_t K, int scheme,
                 const sp_params* params, void* stream) {
  if (!A_host || !B_host || !C_host) { set_error("A, B and C must not be NULL"); return SP_ERR_INVALID_ARG; }
  if (M <= 0 || N <= 0 || K <= 0) { set_error("M, N, K must be positive"); return SP_ERR_INVALID_ARG; }
  if (M >= (1ll << 31) || N >= (1ll << 31) || K >= (1ll << 31)) { set_error("dimension too large"); return SP_ERR_UNSUPPORTED; }
  if (params && params->struct_size != sizeof(sp_params)) {
    set_error("sp_params.struct_size is %u, expected %zu", params->struct_size, sizeof(sp_params));
    return SP_ERR_INVALID_ARG;
  }
  if (params && (params->flags & SP_FLAG_OVERLAP)) {
    set_error("SP_FLAG_OVERLAP is a statement about device buffers the caller manages; sp_gemm_host orders its own copies and kernels");
    return SP_ERR_INVALID_ARG;
  }
  // One call at a time: the staging area, the two copy streams and their events are shared, and the call ends with a
  // synchronisation anyway.  Calls from several host threads queue up here.
  static std::mutex host_call_mu;
  std::lock_guard<std::mutex> host_call_lock(host_call_mu);
  const size_t out_elt = (params && params->out_dtype == 1) ? 4 : 2;
  auto pad = [](size_t b) { return (b + 255) & ~(size_t)255; };
  const size_t a_bytes = (size_t)M * (size_t)K * 2, b_bytes = (size_t)K * (size_t)N * 2, c_bytes = (size_t)M * (size_t)N * out_elt;
  const size_t need = pad(a_bytes) + pad(b_bytes) + pad(c_bytes);
  int dev = 0;
  int rc = current_device(&dev);
  if (rc != SP_OK) return rc;
  char *dA, *dB, *dC;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState* ds = device_state(dev);
    if (ds->staging_bytes < need) {
      if (ds->staging) cudaFree(ds->staging);
      ds->staging = nullptr; ds->staging_bytes = 0;
      SP_CUDA(cudaMalloc(&ds->staging, need));
      ds->staging_bytes = need;
    }
    dA = (char*)ds->staging; dB = dA + pad(a_bytes); dC = dB + pad(b_bytes);
  }
  cudaStream_t st = (cudaStream_t)stream;
  // Row blocks of C are independent: the copy of the next block of A and the copy-out of the previous block of C
  // overlap the compute of the current one (both PCIe directions busy at once).  The copies in are the long pole (A and
  // B together are twice the bytes of C) and the copy-out of a block can only start once that block of A has landed and
  // been multiplied, so C trails A by one block all the way: what is left to do after the last byte of A has arrived is
  // one block's compute and copy-out.  Hence many small blocks (256 rows, more when M is large), not a few large ones
  // (measured at 8192^3: 5.8 ms with 256-row blocks, 5.9-6.0 with 1024 to 2048, 6.5 with 4096; the two copy directions
  // alone, with no compute between them, take 5.4-5.7 ms in the same pipeline because they slow each other down).
  // A caller table describes the whole grid, so it takes the unsplit path.
  int64_t blk = 256;
  while ((M + blk - 1) / blk > kHostChunks) blk *= 2;
  int64_t row_start[kHostChunks + 1];
  int n_chunks = 0;
  for (int64_t r = 0; r < M; r += blk) row_start[n_chunks++] = r;
  row_start[n_chunks] = M;
  const bool split = M >= 4096 && scheme != kCustom;
  // A die-pinned order needs at least one tile per persistent unit; a row block with fewer runs the same order unpinned.
  const bool pinned = params && (params->flags & SP_FLAG_DIE_PINNED);
  sp_params unpinned_params;
  int pin_units = 0, pin_tm = 256, pin_tn = 256;
  if (pinned) {
    unpinned_params = *params;
    unpinned_params.flags &= ~SP_FLAG_DIE_PINNED;
    if (params->tile_m) { pin_tm = params->tile_m; pin_tn = params->tile_n; }
    pin_units = gemm_units(pin_tm, pin_tn, kMaxTiles);
  }
  if (!split) {
    SP_CUDA(cudaMemcpyAsync(dA, A_host, a_bytes, cudaMemcpyHostToDevice, st));
    SP_CUDA(cudaMemcpyAsync(dB, B_host, b_bytes, cudaMemcpyHostToDevice, st));
    rc = gemm_common(dA, dB, dC, M, N, K, scheme, params, stream, nullptr, false);
    if (rc != SP_OK) return rc;
    SP_CUDA(cudaMemcpyAsync(C_host, dC, c_bytes, cudaMemcpyDeviceToHost, st));
    return sp_get_status(stream, nullptr);
  }
  cudaStream_t cin, cout;
  cudaEvent_t* ev;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState* ds = device_state(dev);
    if (!ds->copy_in) {
      SP_CUDA(cudaStreamCreateWithFlags(&ds->copy_in, cudaStreamNonBlocking));
      SP_CUDA(cudaStreamCreateWithFlags(&ds->copy_out, cudaStreamNonBlocking));
      for (auto& e : ds->ev) SP_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    }
    cin = ds->copy_in; cout = ds->copy_out; ev = ds->ev;
  }
  cudaEvent_t ev_start = ev[2 * kHostChunks], ev_b = ev[2 * kHostChunks + 1], ev_done = ev[2 * kHostChunks + 2];
  SP_CUDA(cudaEventRecord(ev_start, st));                 // the copies start after what is already queued on `stream`
  SP_CUDA(cudaStreamWaitEvent(cin, ev_start, 0));
  SP_CUDA(cudaStreamWaitEvent(cout, ev_start, 0));
  SP_CUDA(cudaMemcpyAsync(dB, B_host, b_bytes, cudaMemcpyHostToDevice, cin));
  SP_CUDA(cudaEventRecord(ev_b, cin));
  for (int i = 0; i < n_chunks; ++i) {
    const int64_t r0 = row_start[i], nr = row_start[i + 1] - r0;
    SP_CUDA(cudaMemcpyAsync(dA + (size_t)r0 * K * 2, (const char*)A_host + (size_t)r0 * K * 2, (size_t)nr * K * 2,
                            cudaMemcpyHostToDevice, cin));
    SP_CUDA(cudaEventRecord(ev[i], cin));
  }
  SP_CUDA(cudaStreamWaitEvent(st, ev_b, 0));
  for (int i = 0; i < n_chunks; ++i) {
    const int64_t r0 = row_start[i], nr = row_start[i + 1] - r0;
    SP_CUDA(cudaStreamWaitEvent(st, ev[i], 0));
    const sp_params* pb = params;
    if (pinned && (pin_units <= 0 || sp_tile_count(nr, N, pin_tm, pin_tn) < pin_units)) pb = &unpinned_params;
    rc = gemm_common(dA + (size_t)r0 * K * 2, dB, dC + (size_t)r0 * N * out_elt, nr, N, K, scheme, pb, stream, nullptr, false);
    if (rc != SP_OK) break;
    SP_CUDA(cudaEventRecord(ev[kHostChunks + i], st));
    SP_CUDA(cudaStreamWaitEvent(cout, ev[kHostChunks + i], 0));
    SP_CUDA(cudaMemcpyAsync((char*)C_host + (size_t)r0 * N * out_elt, dC + (size_t)r0 * N * out_elt, (size_t)nr * N * out_elt,
                            cudaMemcpyDeviceToHost, cout));
  }
  SP_CUDA(cudaEventRecord(ev_done, cout));
  SP_CUDA(cudaStreamWaitEvent(st, ev_done, 0));
  if (rc != SP_OK) { cudaStreamSynchronize(cin); cudaStreamSynchronize(st); return rc; }
  SP_CUDA(cudaStreamSynchronize(cin));
  return sp_get_status(stream, nullptr);
}

int sp_transpose(const void* in, void* out, int64_t M, int64_t N, int scheme, const sp_params* params, void* stream) {
  if (!in || !out) { set_error("in and out must not be NULL"); return SP_ERR_INVALID_ARG; }
  if (M <= 0 || N <= 0) { set_error("M and N must be positive"); return SP_ERR_INVALID_ARG; }
  if (M >= (1ll << 31) || N >= (1ll << 31)) { set_error("dimension too large"); return SP_ERR_UNSUPPORTED; }
  if (((uintptr_t)in | (uintptr_t)out) & 15u) { set_error("in and out must be 16-byte aligned"); return SP_ERR_ALIGNMENT; }
  if ((M % 8) != 0 || (N % 8) != 0) { set_error("M and N must be multiples of 8 (16-byte row pitch)"); return SP_ERR_ALIGNMENT; }
  if (in == out) { set_error("in-place transposition is not supported"); return SP_ERR_INVALID_ARG; }
  Sched sched;
  int rc = resolve_sched(M, N, SP_TRANSPOSE_TILE, SP_TRANSPOSE_TILE, scheme, params, &sched);
  if (rc != SP_OK) return rc;
  std::vector<int32_t> host_perm;
  if (scheme == kCustom || !already_validated(sched)) {
    rc = build_perm_host(sched, params ? params->custom_perm : nullptr, host_perm);
    if (rc != SP_OK) return rc;
    if (scheme != kCustom) remember_validated(sched);
  }
  int dev = 0;
  rc = current_device(&dev);
  if (rc != SP_OK) return rc;
  std::lock_guard<std::mutex> lock(g_mu);
  DeviceState* ds = device_state(dev);
  rc = get_status_word(ds);
  if (rc != SP_OK) return rc;
  const int32_t* perm_dev = nullptr;
  if (sched.use_table) {
    rc = get_table(ds, sched, host_perm, scheme == kCustom, (cudaStream_t)stream, &perm_dev);
    if (rc != SP_OK) return rc;
  }
  return launch_transpose(in, out, M, N, sched, perm_dev, ds->status, (cudaStream_t)stream);
}

int sp_stencil2d(const void* in, void* out, int64_t M, int64_t N, float c_center, float c_neighbor, int scheme,
                 const sp_params* params, void* stream) {
  if (!in || !out) { set_error("in and out must not be NULL"); return SP_ERR_INVALID_ARG; }
  if (M <= 0 || N <= 0) { set_error("M and N must be positive"); return SP_ERR_INVALID_ARG; }
  if (M >= (1ll << 31) - 256 || N >= (1ll << 31) - 256) { set_error("dimension too large"); return SP_ERR_UNSUPPORTED; }
  if (((uintptr_t)in | (uintptr_t)out) & 15u) { set_error("in and out must be 16-byte aligned"); return SP_ERR_ALIGNMENT; }
  if ((N % 4) != 0) { set_error("N must be a multiple of 4 (16-byte row pitch)"); return SP_ERR_ALIGNMENT; }
  if (in == out) { set_error("the sweep is not in place: out must not overlap in"); return SP_ERR_INVALID_ARG; }
  if (!(c_center == c_center) || !(c_neighbor == c_neighbor)) { set_error("coefficients must not be NaN"); return SP_ERR_INVALID_ARG; }
  Sched sched;
  int rc = resolve_sched(M, N, SP_STENCIL_TILE_M, SP_STENCIL_TILE_N, scheme, params, &sched);
  if (rc != SP_OK) return rc;
  std::vector<int32_t> host_perm;
  if (scheme == kCustom || !already_validated(sched)) {
    rc = build_perm_host(sched, params ? params->custom_perm : nullptr, host_perm);
    if (rc != SP_OK) return rc;
    if (scheme != kCustom) remember_validated(sched);
  }
  int dev = 0;
  rc = current_device(&dev);
  if (rc != SP_OK) return rc;
  std::lock_guard<std::mutex> lock(g_mu);
  DeviceState* ds = device_state(dev);
  rc = get_status_word(ds);
  if (rc != SP_OK) return rc;
  const int32_t* perm_dev = nullptr;
  if (sched.use_table) {
    rc = get_table(ds, sched, host_perm, scheme == kCustom, (cudaStream_t)stream, &perm_dev);
    if (rc != SP_OK) return rc;
  }
  return launch_stencil(in, out, M, N, c_center, c_neighbor, sched, perm_dev, ds->status, (cudaStream_t)stream);
}

// Persistent units sp_gemm would launch for a tile shape: asked of the current device when there is one (parts of
// the pool have SMs fused off), else those of a full B200 (148 SMs, one CTA each).
static int units_or_nominal(int tile_m, int tile_n) {
  int n = 0, dev = 0;
  if (cudaGetDeviceCount(&n) == cudaSuccess && n > 0) {
    if (current_device(&dev) == SP_OK) {
      const int u = gemm_units(tile_m, tile_n, kMaxTiles);
      if (u > 0) return u;
    }
  } else {
    cudaGetLastError();
  }
  return 148 / (tile_m / 128);
}

int sp_softmax(const void* in, void* out, int64_t M, int64_t N, int32_t mode, int scheme, const sp_params* params,
               void* stream) {
  if (!in || !out) { set_error("in and out must not be NULL"); return SP_ERR_INVALID_ARG; }
  if (M <= 0 || N <= 0) { set_error("M and N must be positive"); return SP_ERR_INVALID_ARG; }
  if (M >= (1ll << 31) - 256 || N >= (1ll << 31) - 1024) { set_error("dimension too large"); return SP_ERR_UNSUPPORTED; }
  if (mode != SP_SOFTMAX_SINGLE_PASS && mode != SP_SOFTMAX_TWO_PHASE && mode != SP_SOFTMAX_TWO_PHASE_REVERSED) {
    set_error("unknown softmax mode %d", mode);
    return SP_ERR_INVALID_ARG;
  }
  if (((uintptr_t)in | (uintptr_t)out) & 15u) { set_error("in and out must be 16-byte aligned"); return SP_ERR_ALIGNMENT; }
  if ((N % 4) != 0) { set_error("N must be a multiple of 4 (16-byte row pitch)"); return SP_ERR_ALIGNMENT; }
  if (in == out) { set_error("out must not overlap in"); return SP_ERR_INVALID_ARG; }
  int tile_m = SP_SOFTMAX_TILE_M;
  int64_t tile_n = SP_SOFTMAX_TILE_N;
  if (mode == SP_SOFTMAX_SINGLE_PASS) {
    tile_m = softmax_rows_per_block(N);
    tile_n = N;
    if (tile_m < 1) { set_error("single-pass softmax takes rows of up to 131072 elements (eight 64 KiB buffers of a cluster); use a two-phase mode"); return SP_ERR_UNSUPPORTED; }
  }
  Sched sched;
  int rc = resolve_sched(M, N, tile_m, (int32_t)tile_n, scheme, params, &sched);
  if (rc != SP_OK) return rc;
  std::vector<int32_t> host_perm;
  if (scheme == kCustom || !already_validated(sched)) {
    rc = build_perm_host(sched, params ? params->custom_perm : nullptr, host_perm);
    if (rc != SP_OK) return rc;
    if (scheme != kCustom) remember_validated(sched);
  }
  int dev = 0;
  rc = current_device(&dev);
  if (rc != SP_OK) return rc;
  std::lock_guard<std::mutex> lock(g_mu);
  DeviceState* ds = device_state(dev);
  rc = get_status_word(ds);
  if (rc != SP_OK) return rc;
  const int32_t* perm_dev = nullptr;
  if (sched.use_table) {
    rc = get_table(ds, sched, host_perm, scheme == kCustom, (cudaStream_t)stream, &perm_dev);
    if (rc != SP_OK) return rc;
  }
  float* partial = nullptr;
  if (mode != SP_SOFTMAX_SINGLE_PASS) {
    const size_t need = (size_t)M * (size_t)sched.Tn * 2 * sizeof(float);
    if (ds->softmax_ws_bytes < need) {
      if (ds->softmax_ws) cudaFree(ds->softmax_ws);   // synchronises: no kernel can still be using it
      ds->softmax_ws = nullptr; ds->softmax_ws_bytes = 0;
      SP_CUDA(cudaMalloc(&ds->softmax_ws, need));
      ds->softmax_ws_bytes = need;
    }
    partial = static_cast<float*>(ds->softmax_ws);
  }
  return launch_softmax(in, out, M, N, mode, sched, perm_dev, partial, ds->status, (cudaStream_t)stream);
}

int sp_recommend(int64_t M, int64_t N, int64_t K, int32_t out_dtype, int32_t b_layout, sp_params* params, int* scheme) {
  if (!params || !scheme) { set_error("params and scheme must not be NULL"); return SP_ERR_INVALID_ARG; }
  if (M <= 0 || N <= 0 || K <= 0) { set_error("M, N, K must be positive"); return SP_ERR_INVALID_ARG; }
  if ((out_dtype != 0 && out_dtype != 1) || (b_layout != 0 && b_layout != 1)) { set_error("bad out_dtype / b_layout"); return SP_ERR_INVALID_ARG; }
  // relative throughput of the tile shapes at equal work, from the sustained sweeps at 4096^3 and 8192^3
  static const struct { int tm, tn; double eff; } kTiles[] = {
      {256, 512, 1.00}, {256, 256, 0.97}, {128, 256, 0.89}, {256, 128, 0.75}, {128, 128, 0.67}};
  int best = 0;
  double best_cost = 0;
  for (int i = 0; i < 5; ++i) {
    const int64_t T = ((M + kTiles[i].tm - 1) / kTiles[i].tm) * ((N + kTiles[i].tn - 1) / kTiles[i].tn);
    const int cg = kTiles[i].tm / 128, units = units_or_nominal(kTiles[i].tm, kTiles[i].tn);
    const double waves = (double)((T + units - 1) / units);
    const double cost = waves * kTiles[i].tm * kTiles[i].tn / (cg * kTiles[i].eff);
    if (i == 0 || cost < best_cost) { best = i; best_cost = cost; }   // ties keep the larger tile (listed first)
  }
  memset(params, 0, sizeof *params);
  params->struct_size = sizeof(sp_params);
  params->tile_m = kTiles[best].tm; params->tile_n = kTiles[best].tn;
  params->out_dtype = out_dtype; params->b_layout = b_layout;
  params->group = 1;
  // Order: a wave of U tiles should cover a block of C that is about as tall as it is wide, so that it needs the
  // fewest rows of A and columns of B.  When the operands fit in L2 anyway, or the grid is at most ten tiles wide
  // (tall), plain row-major (column-major) already does that; else bands of eight.
  const double operands = 2.0 * ((double)M * (double)K + (double)K * (double)N);
  const int64_t Tm = (M + params->tile_m - 1) / params->tile_m, Tn = (N + params->tile_n - 1) / params->tile_n;
  // A narrow grid whose operands do not fit in L2 still re-reads the long operand's panels round after round: walking K
  // in alternating directions lets a round start on what the last one left (16384x2048x8192: 494 -> 407 MB of DRAM
  // reads, +1 to +4 % in time), and C stores that give way first keep it there.
  const uint32_t narrow_flags = operands > 64.0 * 1048576.0 ? (SP_FLAG_K_ALTERNATE | SP_FLAG_HINT_C_EVICT_FIRST) : 0u;
  if (operands <= 64.0 * 1048576.0 || Tn <= 10) {
    *scheme = SP_ROW_MAJOR;
    params->flags |= narrow_flags;
  } else if (Tm <= 10) {
    *scheme = SP_COL_MAJOR;
    params->flags |= narrow_flags;
  } else {
    *scheme = params->tile_n == 512 ? SP_GROUP_N : SP_GROUP_M;
    params->group = 8;
    // bands walked serpentine-wise, K in alternating directions, C stores evict_first: 3-5 % over plain bands in the
    // steady state at 8192^3 and beyond (a fifth fewer DRAM reads)
    params->flags |= SP_FLAG_SERPENTINE | SP_FLAG_K_ALTERNATE | SP_FLAG_HINT_C_EVICT_FIRST;
  }
  // Fewer tiles than half the units and a long k extent: the k-split puts the idle units to work (measured 1.5x at
  // 1024x1024x8192).  The sum is then taken in a different order than without the flag.
  const int units = units_or_nominal(params->tile_m, params->tile_n);
  const int64_t kblocks = (K + 63) / 64;
  if (params->tile_n <= 256 && Tm * Tn * 2 <= units && kblocks >= 32) params->flags |= SP_FLAG_STREAM_K;
  return SP_OK;
}

int sp_gemm_units(int32_t tile_m, int32_t tile_n, int64_t T) {
  int dev = 0;
  if (current_device(&dev) != SP_OK) return -1;
  return gemm_units(tile_m, tile_n, T);
}

int sp_probe_dispatch(int32_t n_blocks, int32_t cluster, int32_t* smid_host, uint64_t* start_host) {
  if (n_blocks <= 0 || n_blocks > (1 << 20) || (cluster != 1 && cluster != 2) || (n_blocks % cluster) != 0 ||
      !smid_host || !start_host) {
    set_error("bad probe arguments");
    return SP_ERR_INVALID_ARG;
  }
  int dev = 0;
  int rc = current_device(&dev);
  if (rc != SP_OK) return rc;
  return probe_dispatch(n_blocks, cluster, smid_host, start_host);
}

int sp_probe_topology(int32_t* sm_to_die_host, int32_t* n_sm, float* confidence, uint32_t* lat_host) {
  if (!sm_to_die_host || !n_sm || !confidence) { set_error("bad probe arguments"); return SP_ERR_INVALID_ARG; }
  int dev = 0;
  int rc = current_device(&dev);
  if (rc != SP_OK) return rc;
  return probe_topology(sm_to_die_host, n_sm, confidence, lat_host);
}

int sp_probe_l2_capacity(int32_t n_sizes, const int64_t* sizes_bytes, int32_t half, float* gbps_out) {
  if (n_sizes < 1 || n_sizes > 256 || !sizes_bytes || !gbps_out || half < -1 || half > 1) { set_error("bad probe arguments"); return SP_ERR_INVALID_ARG; }
  int dev = 0;
  int rc = current_device(&dev);
  if (rc != SP_OK) return rc;
  uint32_t mask[8] = {};
  if (half >= 0) {
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState* ds = device_state(dev);
    rc = get_die_map(ds);
    if (rc != SP_OK) return rc;
    for (int i = 0; i < 8; ++i) mask[i] = ds->die_mask[i];
  }
  return probe_l2_capacity(n_sizes, sizes_bytes, half, mask, gbps_out);
}

int sp_selftest_pinned_tickets(int32_t n0, int32_t n1, int32_t arrivals0) {
  if (n0 < 0 || n1 < 0 || arrivals0 < 0 || arrivals0 > n0 + n1 || n0 + n1 > (1 << 20)) { set_error("bad arguments"); return SP_ERR_INVALID_ARG; }
  std::vector<int> taken((size_t)(n0 + n1), 0);
  for (int die = 0; die < 2; ++die) {
    const int arrivals = die ? n0 + n1 - arrivals0 : arrivals0;
    for (int r = 0; r < arrivals; ++r) {
      int d, k;
      pinned_ticket(n0, n1, die, r, d, k);
      if (d < 0 || d > 1 || k < 0 || k >= (d ? n1 : n0)) { set_error("ticket out of range"); return SP_ERR_NOT_BIJECTIVE; }
      taken[(size_t)(d ? n0 + k : k)]++;
    }
  }
  for (int v : taken) if (v != 1) { set_error("a (half, rank) pair was not taken exactly once"); return SP_ERR_NOT_BIJECTIVE; }
  return SP_OK;
}

int sp_selftest_timeout(int32_t timeout_us, int32_t* code, int64_t* waited_us) {
  if (timeout_us < 1 || timeout_us > 1000000 || !code || !waited_us) { set_error("bad self-test arguments"); return SP_ERR_INVALID_ARG; }
  int dev = 0;
  int rc = current_device(&dev);
  if (rc != SP_OK) return rc;
  std::lock_guard<std::mutex> lock(g_mu);
  DeviceState* ds = device_state(dev);
  rc = get_status_word(ds);
  if (rc != SP_OK) return rc;
  return selftest_timeout(ds->status, timeout_us, code, waited_us);
}

int sp_get_status(void* stream, int32_t* detail) {
  int dev = 0;
  int rc = current_device(&dev);
  if (rc != SP_OK) return rc;
  SP_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  std::lock_guard<std::mutex> lock(g_mu);
  DeviceState* ds = device_state(dev);
  int32_t word = 0;
  if (ds->status) {
    SP_CUDA(cudaMemcpy(&word, ds->status, sizeof word, cudaMemcpyDeviceToHost));
    // after an expired wait a die-pinned launch may have left its counters behind: everything back to zero
    if (word != 0) SP_CUDA(cudaMemset(ds->status, 0, (2 + kDieWords * kDiePairs) * sizeof(int32_t)));
  }
  if (detail) *detail = word;
  if (word != 0) { set_error("a device-side wait expired (status word 0x%x)", word); return SP_ERR_TIMEOUT; }
  return SP_OK;
}

const char* sp_last_error(void) { return g_err; }

void sp_shutdown(void) {
  std::lock_guard<std::mutex> lock(g_mu);
  int prev = 0;
  const bool have = cudaGetDevice(&prev) == cudaSuccess;
  for (auto& d : g_devs) {
    if (cudaSetDevice(d.device) != cudaSuccess) continue;
    for (auto& e : d.tables) cudaFree(e.dev);
    d.tables.clear();
    if (d.status) cudaFree(d.status);
    d.status = nullptr;
    if (d.staging) cudaFree(d.staging);
    d.staging = nullptr; d.staging_bytes = 0;
    if (d.softmax_ws) cudaFree(d.softmax_ws);
    d.softmax_ws = nullptr; d.softmax_ws_bytes = 0;
    for (auto& sk : d.sk_spaces) cudaFree(sk.mem);
    d.sk_spaces.clear();
    if (d.copy_in) {
      cudaStreamDestroy(d.copy_in); cudaStreamDestroy(d.copy_out);
      for (auto& e : d.ev) if (e) { cudaEventDestroy(e); e = nullptr; }
      d.copy_in = d.copy_out = nullptr;
    }
  }
  g_devs.clear();
  if (have) cudaSetDevice(prev);
  cudaGetLastError();
}

}  // extern "C"
