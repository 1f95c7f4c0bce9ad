// Persistent, warp-specialised bf16 GEMM for sm_100a whose tile order is a remap of slot ids
// (the paper's swizzle: each block recomputes which output tile it works on).
//
// One persistent unit = one CTA (tile 128 x BN) or a CTA pair (tile 256 x BN, cta_group::2).  BN = 512 is two
// 256-wide MMA tiles that share the A panel (one accumulator each, no double buffering): a quarter less operand
// traffic from L2 per flop, at the price of an epilogue that is not hidden behind the next tile's mainloop.
// Unit u runs slots u, u + units, u + 2*units, ...; slot s computes tile slot_to_tile(s).
//
// Warp roles (192 threads; 384 for BN = 512, where warps 2 and 3 idle so that the epilogue warps start on a warp-group
// boundary and the register file can be re-divided: 72 registers for the issuing group, 216 for the epilogue groups):
//   warp 0         : TMA producer   -- A and B k-blocks into a ring of 128B-swizzled smem stages (whole warp in the
//                                      loop, one elected lane issues)
//   warp 1         : MMA issuer     -- tcgen05.mma, fp32 accumulators in TMEM (two buffers, or two parts of one tile
//                                      for BN = 512); elected lane issues; the warp also owns TMEM alloc / dealloc
//   warps 2..5     : epilogue       -- (4..11 for BN = 512, four per accumulator part) tcgen05.ld, convert, stage 32 rows x 128 bytes per warp in swizzled smem,
//                                      TMA store (full 128-byte rows; ragged edges clipped by the tensor map)
//
// Synchronisation: mbarriers only.  full[s]/empty[s] per smem stage, tmem_full[b]/tmem_empty[b]
// per accumulator buffer.  In pair mode the barriers that feed the MMA issuer live in the
// leader CTA (cluster rank 0); tcgen05.commit multicasts its arrivals to both CTAs.
// Every wait is bounded: after kTimeoutNs, or once another role has given up, the role
// records a code in the status word and leaves; teardown always runs and frees TMEM.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdio.h>
#include <stdlib.h>

#include <mutex>

#include "internal.h"
#include "ptx.cuh"
#include "streamk.cuh"

namespace sp {

constexpr int kBK = 64;          // k extent of one stage: 64 bf16 = one 128-byte swizzle row
constexpr int kUmmaK = 16;       // k extent of one tcgen05.mma with 16-bit inputs
constexpr uint32_t kSmemLimit = 232448;  // 227 KiB opt-in maximum per CTA
constexpr uint32_t kBarrierBytes = 1024;
constexpr int kTmemCols = 512;
constexpr int kClcDepth = 4;     // responses of cluster launch control in flight / not yet read by every role

template <int CG, int BN>
struct Cfg {
  static constexpr int kMmaN = BN > 256 ? 256 : BN;             // N of one tcgen05.mma
  static constexpr int kNT = BN / kMmaN;                        // MMA tiles side by side in one scheduler tile
  static constexpr int kBufs = kNT == 1 ? 2 : 1;                // accumulator buffers of BN columns in the 512 TMEM columns
  static constexpr int kEpiWarps = kNT == 1 ? 4 : 8;            // one per TMEM lane quarter and accumulator part
  // Warps: producer, MMA issuer, then the epilogue warps.  With two MMA tiles the epilogue warps start on a warp-group
  // boundary (warps 2 and 3 idle), so that the register file can be re-divided between the groups (setmaxnreg works
  // per group of four warps): the two issuing warps need few registers, the epilogue warps many.
  static constexpr int kEpi0 = kNT == 1 ? 2 : 4;                // first epilogue warp
  static constexpr int kThreads = 32 * (kEpi0 + kEpiWarps);
  static constexpr int kGroup = 2;                                  // kNT == 2: k-blocks issued part by part at both ends of a tile
  static constexpr int kRegsIssue = 72, kRegsEpilogue = 216;    // kNT == 2: 128 x 72 + 256 x 216 = 64512 registers
  static constexpr int kMmaCols = kMmaN / CG;                   // columns of B one CTA supplies to one MMA
  static constexpr int kBCols = BN / CG;                        // columns of B held by one CTA
  static constexpr uint32_t kABytes = 128 * kBK * 2;            // 128 rows of A
  static constexpr uint32_t kBBytes = kBCols * kBK * 2;
  static constexpr uint32_t kStageBytes = kABytes + kBBytes;
  static constexpr uint32_t kEpiBytes = 4 * 2 * 4096;           // per epilogue warp: two 32-row x 128-byte staging buffers
  static constexpr int kFit = (kSmemLimit - kBarrierBytes - 1024 - kEpiBytes) / kStageBytes;
  static constexpr int kStages = kFit > 8 ? 8 : kFit;
  static constexpr uint32_t kSmemBytes = kStages * kStageBytes + kEpiBytes + kBarrierBytes + 1024;  // + alignment slack
};

struct GemmArgs {
  void* C;
  const int32_t* perm;
  int32_t* status;
  sp_trace_rec* trace;
  int M, N, K;
  int kblocks;
  int units;
  uint32_t b_lbo, b_sbo, b_kstep;  // B operand descriptor strides in bytes
  // Die-pinned scheduling (SP_DIE_SPLIT with SP_FLAG_DIE_PINNED): units on L2 half d run the slots of half d only.
  int pinned;                      // 0: slot s runs on unit s % units
  int half0;                       // number of slots in half 0 (queue boundary)
  int units_on_die[2];             // persistent units per die (all SMs host one CTA each)
  int32_t* die_count;              // five device counters, zero at launch: arrivals on half 0, on half 1, units finished,
                                   // and (SP_FLAG_STEAL) the next ticket of the queue of half 0 and of half 1
  int steal;                       // 1: the slots of each half are handed out by ticket, a unit whose own half is exhausted
                                   //    takes tickets of the other half (pinned must be 1)
  uint32_t die_mask[8];            // bit smid = die of that SM (from the topology probe)
  // Stream-K tail (SP_FLAG_STREAM_K): the last sk.tiles slots are split along k over sk.units units.
  SkPlan sk;
  float* sk_ws;                    // one fp32 partial tile per unit: [unit][cta of the unit][lane quarter][column][lane]
  int32_t* sk_flags;               // one word per (unit, cta, lane quarter): set to sk_epoch once that partial is complete
  int32_t sk_epoch;                // differs from launch to launch on one workspace, so the flags need no clearing
  int overlap;                     // 1: never waits for its predecessor before working (only before exiting)
  int hint_a, hint_b, hint_c;      // L2 eviction priority of A loads, B loads, C stores: 0 none, 1 evict_first, 2 evict_last
  int k_alternate;                 // 1: every other piece of work of a unit walks its k-blocks from the far end (SP_FLAG_K_ALTERNATE)
  int clc;                         // 1: one cluster per tile is launched; running clusters take over the slots of clusters
                                   //    not yet started (cluster launch control) instead of striding through the slots
  Sched sched;
};


// status word: (role << 8) | which wait
enum : int { kRoleProducer = 1, kRoleMma = 2, kRoleEpilogue = 3 };

// (PTX wrappers: ptx.cuh)
// Shared-memory operand descriptor (tcgen05): start address, leading / stride byte offsets
// (all in 16-byte units), descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}

// The same descriptor for another start address: `base` was built for address 0, `addr16` is the byte address >> 4
// (below 2^14: shared memory ends at 227 KiB).  Only the low word changes: one 32-bit add per descriptor in the
// issue loop instead of the full field arithmetic.
__device__ __forceinline__ uint64_t desc_at(uint64_t base, uint32_t addr16) {
  return ((uint64_t)(uint32_t)(base >> 32) << 32) | (uint64_t)((uint32_t)base + addr16);
}

// Instruction descriptor, kind::f16: D fp32, A and B bf16, A K-major, B K- or MN-major.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ int tile_of_slot(const GemmArgs& a, int s) {
  return a.sched.use_table ? __ldg(a.perm + s) : slot_to_tile(a.sched, s);
}

__device__ __forceinline__ uint32_t pack_bf16(uint32_t lo_bits, uint32_t hi_bits) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(lo_bits), __uint_as_float(hi_bits));
  return *reinterpret_cast<const uint32_t*>(&v);
}

// ------------------------------------------------------------------ the kernel
// DYN selects the build that also contains the two dynamic hand-outs of slots (cluster launch control, per-half ticket
// queues with stealing); the static schedules (fixed stride, die-pinned ranks, k-split tail) run the build without
// them, which keeps their code and register pressure out of the default path.
template <int CG, int BN, bool B_NK, bool OUT_F32, bool DYN>
__global__ void __launch_bounds__((Cfg<CG, BN>::kThreads), 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmC, const GemmArgs args) {
  using C = Cfg<CG, BN>;
  constexpr int S = C::kStages;
  constexpr int TILE_M = 128 * CG;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t epi_base = smem_base + S * C::kStageBytes;   // 1024-byte aligned: the store's 128-byte swizzle needs it
  const uint32_t bar_base = epi_base + C::kEpiBytes;
  const uint32_t bar_full = bar_base;              // S barriers
  const uint32_t bar_empty = bar_base + 8 * S;     // S barriers
  const uint32_t bar_tfull = bar_base + 16 * S;    // 2 barriers
  const uint32_t bar_tempty = bar_tfull + 16;      // 2 barriers
  const uint32_t tmem_slot = bar_tempty + 16;      // 4 bytes
  const uint32_t clc_resp = bar_base + 256;        // kClcDepth responses of 16 bytes (cluster launch control)
  const uint32_t clc_full = clc_resp + 16 * kClcDepth, clc_empty = clc_full + 8 * kClcDepth;
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = CG == 1 ? 0u : cluster_ctarank();
  const int unit = blockIdx.x / CG;
  const int T = args.sched.T, Tn = args.sched.Tn;
  const int KB = args.kblocks;

  // A GEMM launched behind this one with SP_FLAG_OVERLAP may be scheduled from now on: its CTAs become resident as
  // ours exit (shared memory admits one CTA per SM).  Without such a successor this is a no-op.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x == 32) { prefetch_tensormap(&tmA); prefetch_tensormap(&tmB); prefetch_tensormap(&tmC); }
  if (threadIdx.x == 0) {
    for (int i = 0; i < S; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar_tfull + 8 * i, 1); mbar_init(bar_tempty + 8 * i, 4 * CG); }
    // a response is read by the producer and the epilogue warps of every CTA of the unit and by the leader's MMA warp
    for (int i = 0; i < kClcDepth; ++i) { mbar_init(clc_full + 8 * i, 1); mbar_init(clc_empty + 8 * i, CG * (1 + C::kEpiWarps) + 1); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc<CG>(tmem_slot, kTmemCols);
    tmem_relinquish<CG>();
  }
  const uint32_t sched_slot = tmem_slot + 8;       // 2 words: die, rank on that die
  if (args.pinned && !args.steal && threadIdx.x == 32 * 2 && rank == 0) {
    // the leader learns which L2 half its SM belongs to and takes the next rank there;
    // both CTAs of the unit read the pair of words after the start-up barrier
    uint32_t smid;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    const int my_die = (int)((args.die_mask[(smid >> 5) & 7] >> (smid & 31)) & 1u);
    const int arrival = atomicAdd(args.die_count + my_die, 1);
    int die_i, rank_i;   // normally (my_die, arrival); re-assigned only if the GPU is shared and placement is uneven
    pinned_ticket(args.units_on_die[0], args.units_on_die[1], my_die, arrival, die_i, rank_i);
    const uint32_t die = (uint32_t)die_i, r = (uint32_t)rank_i;
#pragma unroll
    for (uint32_t c = 0; c < (uint32_t)CG; ++c) {
      const uint32_t dst = CG == 1 ? sched_slot : mapa(sched_slot, c);
      asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(dst), "r"(die) : "memory");
      asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(dst + 4), "r"(r) : "memory");
    }
  }
  tcgen05_fence_before();
  unit_sync<CG>();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;
  // whole tiles of this unit: slots s_first, s_first + s_step, ... below s_end; then its segments of the stream-K tail
  int s_first = unit, s_step = args.units, s_end = args.sk.first_slot;
  if (args.pinned && !args.steal) {
    const uint32_t die = tmem_slot_ptr[2], r = tmem_slot_ptr[3];
    s_step = args.units_on_die[die];
    s_first = (die ? args.half0 : 0) + (int)r;
    s_end = die ? T : args.half0;
  }
  const int n_whole = s_first < s_end ? (s_end - s_first + s_step - 1) / s_step : 0;
  // The first tile of a fixed schedule does not depend on the kernel before this one: the producer warp decodes it now
  // (arithmetic orders; a table lives in global memory), off the path that starts when that kernel has finished.  For a
  // grid of a few tiles the chain of integer divisions is a few per cent of the launch.
  int t_first = -1;
  if (warp == 0 && !args.sched.use_table && n_whole > 0 && !(DYN && (args.steal || args.clc))) t_first = slot_to_tile(args.sched, s_first);
  // Every launch is made with programmatic stream serialisation: the set-up above may run while the kernel before
  // this one on the stream is still finishing (its CTAs leaving free the SMs ours start on).  From here on global
  // memory is touched, so an ordinary launch now waits until that kernel has completed and its writes are visible;
  // a launch declared independent of it (SP_FLAG_OVERLAP) goes straight on and waits only before it exits.
  if (!args.overlap) asm volatile("griddepcontrol.wait;" ::: "memory");

  const int n_items = n_whole + sk_segments(args.sk, unit, KB);
  // The i-th piece of work of this unit; slot < 0 when there is none.  Called by whole warps, every role with its own
  // counter.  With cluster launch control the first tile is the cluster's own and every further one comes from a
  // response the leader's producer warp asked for one tile earlier (ring of kClcDepth responses, written to every CTA
  // of the unit by the hardware; a reader hands the entry back on the leader's barrier).
  auto work_at = [&](int i, int wait_code) -> Work {
    Work w; w.k0 = 0; w.k1 = KB; w.kind = kWorkFull; w.slot = -1;
    if (DYN && args.steal) {
      // every item comes from the ring: the leader's producer warp took a ticket for it and wrote the slot (or -1)
      // into the entry of every CTA of the unit
      const int e = i % kClcDepth;
      bool oks = mbar_wait_cluster_acquire(clc_full + 8 * e, (uint32_t)(i / kClcDepth) & 1u, args.status, wait_code);
      oks = __all_sync(0xffffffffu, oks);
      int got = -1;
      if (oks) got = *reinterpret_cast<volatile int32_t*>(smem_raw + (clc_resp + 16 * e - smem_u32(smem_raw)));
      __syncwarp();
      if (oks && elect_one()) mbar_arrive_cluster(CG == 1 ? clc_empty + 8 * e : mapa(clc_empty + 8 * e, 0));
      w.slot = got;
      return w;
    }
    if (DYN && args.clc) {
      if (i == 0) { w.slot = unit; return w; }
      const int e = (i - 1) % kClcDepth;
      bool okc = mbar_wait(clc_full + 8 * e, (uint32_t)((i - 1) / kClcDepth) & 1u, args.status, wait_code);
      okc = __all_sync(0xffffffffu, okc);
      uint32_t valid = 0, first_cta = 0;
      if (okc) clc_decode(clc_resp + 16 * e, valid, first_cta);
      __syncwarp();
      if (okc && elect_one()) mbar_arrive_cluster(CG == 1 ? clc_empty + 8 * e : mapa(clc_empty + 8 * e, 0));
      if (okc && valid) w.slot = (int)(first_cta / CG);
      return w;
    }
    if (i < n_whole) { w.slot = s_first + i * s_step; return w; }
    if (i < n_items) return sk_segment(args.sk, unit, i - n_whole, KB);
    return w;
  };

  if (warp < C::kEpi0) {
  if constexpr (C::kNT == 2) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(C::kRegsIssue));
  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    // The whole warp walks the loop (uniform control flow, uniform operands); one elected
    // lane issues the copies.
    {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const bool hinted = (args.hint_a | args.hint_b) != 0;
      const uint64_t pol_a = l2_policy(args.hint_a), pol_b = l2_policy(args.hint_b);
      auto load_a = [&](uint32_t dst, int x, int y, uint32_t bar) {
        if (hinted) tma_load_2d_hint<CG>(dst, &tmA, x, y, bar, pol_a); else tma_load_2d<CG>(dst, &tmA, x, y, bar);
      };
      auto load_b = [&](uint32_t dst, int x, int y, uint32_t bar) {
        if (hinted) tma_load_2d_hint<CG>(dst, &tmB, x, y, bar, pol_b); else tma_load_2d<CG>(dst, &tmB, x, y, bar);
      };
      int my_die = 0;
      if (DYN && args.steal) {
        uint32_t smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        my_die = (int)((args.die_mask[(smid >> 5) & 7] >> (smid & 31)) & 1u);
      }
      for (int item = 0; ok; ++item) {
        if (DYN && args.steal && rank == 0) {
          // Take the next ticket of this unit's own half, or, once that queue is empty, of the other half; publish the
          // slot to every CTA of the unit.  Taken only now, when the loads of the previous tile have all been issued,
          // so a unit never holds a tile it is not about to start.
          const int e = item % kClcDepth;
          if (item >= kClcDepth) {
            ok = mbar_wait(clc_empty + 8 * e, (uint32_t)(item / kClcDepth - 1) & 1u, args.status, (kRoleProducer << 8) | 5);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
          }
          if (elect_one()) {
            const int size0 = args.half0, size1 = T - args.half0;
            int slot = -1;
            int t = atomicAdd(args.die_count + 3 + my_die, 1);
            if (t < (my_die ? size1 : size0)) slot = (my_die ? size0 : 0) + t;
            else {
              t = atomicAdd(args.die_count + 3 + (my_die ^ 1), 1);
              if (t < (my_die ? size0 : size1)) slot = (my_die ? 0 : size0) + t;
            }
#pragma unroll
            for (uint32_t c = 0; c < (uint32_t)CG; ++c) {
              const uint32_t dst = CG == 1 ? clc_resp + 16 * e : mapa(clc_resp + 16 * e, c);
              asm volatile("st.shared::cluster.s32 [%0], %1;" ::"r"(dst), "r"(slot) : "memory");
              mbar_arrive_cluster(CG == 1 ? clc_full + 8 * e : mapa(clc_full + 8 * e, c));
            }
          }
          __syncwarp();
        }
        const Work wk = work_at(item, (kRoleProducer << 8) | 4);
        if (wk.slot < 0) break;
        const int s = wk.slot;
        if (DYN && args.clc) {
          // ask for the tile after this one: every CTA arms its own barrier for the 16 bytes the hardware will write
          // to it; the leader first makes sure every reader has handed the entry back, then issues the request
          const int e = item % kClcDepth;
          if (rank == 0 && item >= kClcDepth) {
            ok = mbar_wait(clc_empty + 8 * e, (uint32_t)(item / kClcDepth - 1) & 1u, args.status, (kRoleProducer << 8) | 5);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
          }
          if (elect_one()) {
            mbar_arrive_expect_tx(clc_full + 8 * e, 16);
            if (rank == 0) clc_try_cancel<CG>(clc_resp + 16 * e, clc_full + 8 * e);
          }
          __syncwarp();
        }
        const int t = (item == 0 && t_first >= 0) ? t_first : tile_of_slot(args, s);
        const int tm = t / Tn, tn = t - tm * Tn;
        const int row0 = tm * TILE_M + (int)rank * 128;
        const int col0 = tn * BN + (int)rank * C::kMmaCols;        // + c * kMmaN for the c-th MMA tile
        const bool tracing = args.trace != nullptr && rank == 0 && wk.kind != kWorkContrib;   // a split tile is traced by the piece that stores it
        uint32_t waited = 0;
        // SP_FLAG_K_ALTERNATE: odd items of a unit load their k-blocks in descending order.  The tiles of one round run in
        // step, so the round that follows starts on the k-range its predecessor touched last, which is what L2 still holds.
        const bool k_desc = args.k_alternate && (item & 1);
        if (tracing && lane == 0) {
          sp_trace_rec* rec = args.trace + s;
          uint32_t smid;
          asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
          rec->slot = s; rec->tile = t; rec->smid = (int)smid; rec->unit = unit; rec->t_begin = globaltimer();
        }
        for (int kb = wk.k0; kb < wk.k1; ++kb) {
          ok = mbar_wait_timed(bar_empty + 8 * stage, phase ^ 1u, args.status, (kRoleProducer << 8) | 1, tracing, &waited);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          const uint32_t full_local = bar_full + 8 * stage;
          const uint32_t full_leader = CG == 1 ? full_local : mapa(full_local, 0);
          const uint32_t sa = smem_base + stage * C::kStageBytes;
          const uint32_t sb = sa + C::kABytes;
          const int k_elem = (k_desc ? wk.k0 + wk.k1 - 1 - kb : kb) * kBK;
          if (elect_one()) {
            if (rank == 0) mbar_arrive_expect_tx(full_local, CG * C::kStageBytes);
            load_a(sa, k_elem, row0, full_leader);
            if constexpr (B_NK) {
#pragma unroll
              for (int c = 0; c < C::kNT; ++c)
                load_b(sb + c * (C::kMmaCols * kBK * 2), k_elem, col0 + c * C::kMmaN, full_leader);
            } else {
#pragma unroll
              for (int j = 0; j < C::kBCols / 64; ++j) {   // boxes of 64 columns, MMA tile by MMA tile
                constexpr int per = C::kMmaCols / 64;
                load_b(sb + j * (64 * kBK * 2), col0 + (j / per) * C::kMmaN + (j % per) * 64, k_elem, full_leader);
              }
            }
          }
          __syncwarp();
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
        if (tracing && lane == 0) args.trace[s].load_wait_stage = waited;
      }
      // tail: every stage handed out must have been released, so that no commit arrival
      // (or, after a failure, no copy) is still in flight towards this CTA when it exits
      for (int i = 0; i < S && ok; ++i) {
        ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, args.status, (kRoleProducer << 8) | 2);
        ok = __all_sync(0xffffffffu, ok);
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
      if (!ok) {
        const unsigned long long t0 = globaltimer();
        while (globaltimer() - t0 < 1000000ull) __nanosleep(1000);  // let copies in flight land
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (leader CTA only)
    // Whole warp in the loop, one elected lane issues: descriptors stay warp-uniform values.
    if (rank == 0) {
      constexpr uint32_t idesc = make_idesc(TILE_M, C::kMmaN, !B_NK);
      const uint64_t da0 = smem_desc(0, 16, 1024), db0 = smem_desc(0, args.b_lbo, args.b_sbo);
      const uint32_t b_kstep16 = args.b_kstep >> 4;
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      // Accumulator parts.  One MMA tile per scheduler tile: one part, alternating between two TMEM buffers.
      // Two MMA tiles (BN = 512): two parts, each with its own pair of barriers, so the epilogue can drain the
      // first while the second is still being computed, and the next tile can start on the first part while the
      // second is being drained.
      for (; ok; ++it) {
        const Work wk = work_at(it, (kRoleMma << 8) | 4);
        if (wk.slot < 0) break;
        const int s = wk.slot;
        const int buf = it % C::kBufs;
        const uint32_t use = C::kNT == 1 ? ((uint32_t)(it / C::kBufs) & 1u) : ((uint32_t)it & 1u);
        const bool tracing = args.trace != nullptr && wk.kind != kWorkContrib;
        uint32_t wait_acc = 0, wait_data = 0;
        if (tracing && lane == 0) args.trace[s].t_mma_begin = globaltimer();
        if constexpr (C::kNT == 2) {
          // K-blocks are issued in groups: the first kGroup and the last kGroup k-blocks of a tile as a group, the rest one
          // by one.  Inside a group the first MMA tile's MMAs come before the second's (each k-block as soon as it has
          // landed).  The first accumulator part is then complete kGroup x 512 cycles of MMAs before the second, and the
          // next tile starts on it equally early: the epilogue warps of one part drain it (about 1800 cycles) while the
          // tensor pipe works on the other.  The body keeps the full look-ahead of the ring; a group holds kGroup of its
          // stages until the second part has used them.  Groups of 3 and 4 were measured: 1 % slower than 2, with the
          // same tensor-pipe activity (the stages a longer group holds back cost what its longer cover gains).
          constexpr int G = C::kGroup;
          int kb = 0;
          while (kb < KB && ok) {
            const bool grouped = KB >= 2 * G && (kb == 0 || kb == KB - G);
            const int g = grouped ? G : 1;
            uint32_t st[G];
#pragma unroll
            for (int c = 0; c < 2; ++c) {
              if (kb == 0) {                                        // the part must have been drained by the previous tile's epilogue
                ok = mbar_wait_timed(bar_tempty + 8 * c, use ^ 1u, args.status, (kRoleMma << 8) | 1, tracing, &wait_acc);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tcgen05_fence_after();
              }
#pragma unroll
              for (int i = 0; i < G; ++i) {
                if (i >= g) break;
                if (c == 0) {                                       // the first part takes each k-block as soon as it has landed
                  ok = mbar_wait_timed(bar_full + 8 * stage, phase, args.status, (kRoleMma << 8) | 2, tracing, &wait_data);
                  ok = __all_sync(0xffffffffu, ok);
                  if (!ok) break;
                  tcgen05_fence_after();
                  st[i] = (uint32_t)stage;
                  if (++stage == S) { stage = 0; phase ^= 1u; }
                }
                if (elect_one()) {
                  const uint32_t sa = smem_base + st[i] * C::kStageBytes;
                  const uint32_t sb = sa + C::kABytes + (uint32_t)(c * C::kMmaCols * kBK * 2);
#pragma unroll
                  for (int k = 0; k < kBK / kUmmaK; ++k) {
                    const uint64_t da = desc_at(da0, (sa >> 4) + k * (kUmmaK * 2 / 16));
                    const uint64_t db = desc_at(db0, (sb >> 4) + k * b_kstep16);
                    umma_bf16<CG>(tmem_base + (uint32_t)(c * C::kMmaN), da, db, idesc, (uint32_t)(((kb + i) | k) != 0));
                  }
                  if (c == 1) umma_commit<CG>(bar_empty + 8 * st[i]);          // both parts have used the stage
                  if (kb + i + 1 == KB) umma_commit<CG>(bar_tfull + 8 * c);     // this part is complete
                }
                __syncwarp();
              }
              if (!ok) break;
            }
            if (!ok) break;
            kb += g;
          }
        } else {
        for (int kb = wk.k0; kb < wk.k1 && ok; ++kb) {        // all k-blocks of the tile, or this unit's segment of them
          ok = mbar_wait_timed(bar_full + 8 * stage, phase, args.status, (kRoleMma << 8) | 2, tracing, &wait_data);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tcgen05_fence_after();
          const uint32_t sa = smem_base + stage * C::kStageBytes;
          const uint32_t sb = sa + C::kABytes;
#pragma unroll
          for (int c = 0; c < C::kNT; ++c) {
            const int part = C::kNT == 1 ? buf : c;
            if (kb == wk.k0) {                   // the part must have been drained by the epilogue of its previous use
              ok = mbar_wait_timed(bar_tempty + 8 * part, use ^ 1u, args.status, (kRoleMma << 8) | 1, tracing, &wait_acc);
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) break;
              tcgen05_fence_after();
            }
            const uint32_t d_tmem = tmem_base + (uint32_t)(C::kNT == 1 ? buf * BN : c * C::kMmaN);
            if (elect_one()) {
#pragma unroll
              for (int k = 0; k < kBK / kUmmaK; ++k) {
                const uint64_t da = desc_at(da0, (sa >> 4) + k * (kUmmaK * 2 / 16));
                const uint64_t db = desc_at(db0, ((sb + c * (C::kMmaCols * kBK * 2)) >> 4) + k * b_kstep16);
                umma_bf16<CG>(d_tmem, da, db, idesc, (uint32_t)(kb > wk.k0 || k != 0));
              }
              if (kb == wk.k1 - 1) umma_commit<CG>(bar_tfull + 8 * part);   // this part is complete
            }
            __syncwarp();
          }
          if (!ok) break;
          if (elect_one()) umma_commit<CG>(bar_empty + 8 * stage);
          __syncwarp();
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
        }
        if (tracing && lane == 0) {
          sp_trace_rec* rec = args.trace + s;
          rec->mma_wait_data = wait_data; rec->mma_wait_acc = wait_acc; rec->t_mma_issued = globaltimer();
        }
      }
    }
    __syncwarp();
  }
  } else {
    // ---------------------------------------------------------------- epilogue
    if constexpr (C::kNT == 2) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(C::kRegsEpilogue));
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, 32*quarter + 32) are this warp's
    auto store_c = [&](uint32_t src, int x, int y) {   // issued by one lane
      if (args.hint_c) tma_store_2d_hint(&tmC, src, x, y, l2_policy(args.hint_c)); else tma_store_2d(&tmC, src, x, y);
    };
    if constexpr (C::kNT == 2) {
      // Two MMA tiles per scheduler tile: no second accumulator buffer hides this epilogue.  Four warps serve each
      // accumulator part.  A warp empties its 32 lanes x 256 columns into registers (packed bf16), hands the part back
      // to the MMA issuer at once, and only then stages and stores (one 4 KiB slice per warp), which overlaps the
      // mainloop that has already resumed; the other part's warps are never held up by these stores.
      const int c = (warp - C::kEpi0) >> 2;                        // the part this warp serves
      const uint32_t slice = epi_base + (uint32_t)((warp - C::kEpi0) * 4096);
      const uint32_t rowaddr = slice + (uint32_t)lane * 128u;
      const uint32_t sw = (uint32_t)lane & 7u;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * C::kMmaN);
      int it2 = 0;
      bool ok2 = true;
      for (; ok2; ++it2) {
        const int s = work_at(it2, (kRoleEpilogue << 8) | 4).slot;
        if (s < 0) break;
        const int t = tile_of_slot(args, s);
        const int tm = t / Tn, tn = t - tm * Tn;
        const uint32_t use = (uint32_t)it2 & 1u;
        const int row0 = tm * TILE_M + (int)rank * 128 + quarter * 32;
        const int col_base = tn * BN + c * C::kMmaN;
        uint32_t wait_epi = 0;
        ok2 = mbar_wait_timed(bar_tfull + 8 * c, use, args.status, (kRoleEpilogue << 8) | 1, args.trace != nullptr, &wait_epi);
        ok2 = __all_sync(0xffffffffu, ok2);
        if (!ok2) break;
        tcgen05_fence_after();
        if constexpr (!OUT_F32) {
          uint32_t pk[C::kMmaN / 2];
#pragma unroll
          for (int q = 0; q < C::kMmaN / 64; ++q) {                  // two read-outs of 32 columns in flight per round trip
            uint32_t v[32], w[32];
            tmem_ld_32x32b_x32(taddr + (uint32_t)(q * 64), v);
            tmem_ld_32x32b_x32(taddr + (uint32_t)(q * 64 + 32), w);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              pk[q * 32 + j] = pack_bf16(v[2 * j], v[2 * j + 1]);
              pk[q * 32 + 16 + j] = pack_bf16(w[2 * j], w[2 * j + 1]);
            }
          }
          tcgen05_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(mapa(bar_tempty + 8 * c, 0));
#pragma unroll
          for (int q = 0; q < C::kMmaN / 64; ++q) {
            if (lane == 0) bulk_wait_read_0();                      // the slice's previous store has read it
            __syncwarp();
#pragma unroll
            for (uint32_t j = 0; j < 8; ++j)
              st_shared_16(rowaddr + ((j ^ sw) << 4), pk[q * 32 + 4 * j], pk[q * 32 + 4 * j + 1], pk[q * 32 + 4 * j + 2],
                           pk[q * 32 + 4 * j + 3]);
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              const int col = col_base + q * 64;
              if (row0 < args.M && col < args.N) store_c(slice, col, row0);
              bulk_commit();
            }
          }
        } else {
          // fp32 output: 256 columns do not fit in registers; chunk by chunk, the part is released at the end
#pragma unroll 1
          for (int q = 0; q < C::kMmaN / 32; ++q) {
            uint32_t v[32];
            tmem_ld_32x32b_x32(taddr + (uint32_t)(q * 32), v);
            tmem_ld_wait();
            if (lane == 0) bulk_wait_read_0();
            __syncwarp();
#pragma unroll
            for (uint32_t j = 0; j < 8; ++j)
              st_shared_16(rowaddr + ((j ^ sw) << 4), v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              const int col = col_base + q * 32;
              if (row0 < args.M && col < args.N) store_c(slice, col, row0);
              bulk_commit();
            }
          }
          tcgen05_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(mapa(bar_tempty + 8 * c, 0));
        }
        if (lane == 0 && args.trace && rank == 0 && warp == C::kEpi0 + 4) {   // the second part finishes last
          args.trace[s].t_end = globaltimer();
          args.trace[s].epi_wait_acc = wait_epi;
        }
      }
      if (lane == 0) bulk_wait_all();
      __syncwarp();
    } else {
    int it = 0;
    int chunk = 0;                 // staging buffers alternate per stored chunk, across tiles
    bool ok = true;
    for (; ok; ++it) {
      const Work wk = work_at(it, (kRoleEpilogue << 8) | 4);
      if (wk.slot < 0) break;
      const int s = wk.slot;
      const int t = tile_of_slot(args, s);
      const int tm = t / Tn, tn = t - tm * Tn;
      const int buf = it % C::kBufs;
      const uint32_t use = C::kNT == 1 ? ((uint32_t)(it / C::kBufs) & 1u) : ((uint32_t)it & 1u);
      uint32_t wait_epi = 0;
      const int row0 = tm * TILE_M + (int)rank * 128 + quarter * 32;   // first of this warp's 32 rows
      constexpr int kChunkCols = OUT_F32 ? 32 : 64;                    // 128 bytes of output per row
      constexpr int kPartCols = C::kNT == 1 ? BN : C::kMmaN;
#pragma unroll 1
      for (int c = 0; c < C::kNT && ok; ++c) {                         // accumulator parts, in the order they complete
        const int part = C::kNT == 1 ? buf : c;
        // stream-K workspace of (unit u, this CTA, this lane quarter), in 16-byte units: [column / 4][lane]; one warp
        // instruction writes (and later reads) 512 contiguous bytes
        auto ws_of = [&](int u) -> float4* {
          return reinterpret_cast<float4*>(args.sk_ws) + ((((size_t)u * CG + rank) * 4 + (size_t)quarter) * (BN / 4)) * 32 + lane;
        };
        constexpr int kPf = kChunkCols / 4;     // 16-byte units of one chunk of this thread's row
        float4 pf[kPf];                         // owner segments: the nearest contributor's chunk, fetched one chunk ahead
        int n_src = 0;                          // partials to add: those of units unit-1 ... unit-n_src
        if (wk.kind == kWorkOwner) {
          // the contributors finished these pieces at the start of their tails, long before this unit's own MMAs end:
          // the flags are checked and the first chunk is fetched while the accumulator is still being computed
          n_src = sk_contributors(args.sk, unit, s, KB);
          for (int i = 1; i <= n_src && ok; ++i) {
            bool okf = true;
            if (lane == 0)
              okf = flag_wait(args.sk_flags + ((unit - i) * CG + (int)rank) * 4 + quarter, args.sk_epoch, args.status, (kRoleEpilogue << 8) | 3);
            ok = __all_sync(0xffffffffu, okf);
          }
          if (!ok) break;
          __syncwarp();
          __threadfence();
          const float4* src = ws_of(unit - 1);
#pragma unroll
          for (int j = 0; j < kPf; ++j) pf[j] = __ldcg(src + j * 32);
        }
        ok = mbar_wait_timed(bar_tfull + 8 * part, use, args.status, (kRoleEpilogue << 8) | 1, args.trace != nullptr, &wait_epi);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tcgen05_fence_after();
        const int col_base = tn * BN + c * kPartCols;
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(C::kNT == 1 ? buf * BN : c * C::kMmaN);
        if (wk.kind == kWorkContrib) {
          // a segment that does not finish its tile: the raw fp32 partial goes to the workspace, then the flag goes up
          float4* dst = ws_of(unit);
#pragma unroll 1
          for (int q = 0; q < kPartCols / 32; ++q) {
            uint32_t v[32];
            tmem_ld_32x32b_x32(taddr + (uint32_t)(q * 32), v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 8; ++j)
              __stcg(dst + (size_t)(q * 8 + j) * 32, make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                                 __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3])));
          }
          tcgen05_fence_before();
          __threadfence();
          __syncwarp();
          if (lane == 0) {
            const uint32_t te = bar_tempty + 8 * part;
            mbar_arrive_cluster(CG == 1 ? te : mapa(te, 0));
            st_release_gpu(args.sk_flags + (unit * CG + (int)rank) * 4 + quarter, args.sk_epoch);
          }
          continue;
        }
        {
#pragma unroll 1
        for (int q = 0; q < kPartCols / kChunkCols; ++q, ++chunk) {
          uint32_t v[32], w[32];
          tmem_ld_32x32b_x32(taddr + (uint32_t)(q * kChunkCols), v);
          if constexpr (!OUT_F32) tmem_ld_32x32b_x32(taddr + (uint32_t)(q * kChunkCols + 32), w);
          tmem_ld_wait();
          if (n_src > 0) {
            // fixed order of the sum: own accumulator, then units unit-1, unit-2, ...
            auto add16 = [&](int j, const float4& a) {
              uint32_t* d = (OUT_F32 || j < 8) ? &v[4 * j] : &w[4 * (j - 8)];
              d[0] = __float_as_uint(__uint_as_float(d[0]) + a.x); d[1] = __float_as_uint(__uint_as_float(d[1]) + a.y);
              d[2] = __float_as_uint(__uint_as_float(d[2]) + a.z); d[3] = __float_as_uint(__uint_as_float(d[3]) + a.w);
            };
#pragma unroll
            for (int j = 0; j < kPf; ++j) add16(j, pf[j]);
#pragma unroll 1
            for (int i = 2; i <= n_src; ++i) {
              const float4* src = ws_of(unit - i) + (size_t)(q * kPf) * 32;
#pragma unroll
              for (int j = 0; j < kPf; ++j) add16(j, __ldcg(src + j * 32));
            }
            if (q + 1 < kPartCols / kChunkCols) {        // next chunk's fetch overlaps this chunk's staging and store
              const float4* src = ws_of(unit - 1) + (size_t)((q + 1) * kPf) * 32;
#pragma unroll
              for (int j = 0; j < kPf; ++j) pf[j] = __ldcg(src + j * 32);
            }
          }
          // the buffer used two chunks ago must have been read by its store before it is overwritten
          if (chunk >= 2) {
            if (lane == 0) bulk_wait_read_1();
            __syncwarp();
          }
          const uint32_t slice = epi_base + (uint32_t)((warp - C::kEpi0) * 8192 + (chunk & 1) * 4096);
          const uint32_t rowaddr = slice + (uint32_t)lane * 128u;
          const uint32_t sw = (uint32_t)lane & 7u;                     // 128-byte swizzle: 16-byte unit j of row r sits at j ^ (r % 8)
          if constexpr (OUT_F32) {
#pragma unroll
            for (uint32_t j = 0; j < 8; ++j)
              st_shared_16(rowaddr + ((j ^ sw) << 4), v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
          } else {
#pragma unroll
            for (uint32_t j = 0; j < 4; ++j) {
              st_shared_16(rowaddr + ((j ^ sw) << 4), pack_bf16(v[8 * j], v[8 * j + 1]), pack_bf16(v[8 * j + 2], v[8 * j + 3]),
                           pack_bf16(v[8 * j + 4], v[8 * j + 5]), pack_bf16(v[8 * j + 6], v[8 * j + 7]));
              st_shared_16(rowaddr + (((j + 4) ^ sw) << 4), pack_bf16(w[8 * j], w[8 * j + 1]), pack_bf16(w[8 * j + 2], w[8 * j + 3]),
                           pack_bf16(w[8 * j + 4], w[8 * j + 5]), pack_bf16(w[8 * j + 6], w[8 * j + 7]));
            }
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            const int col = col_base + q * kChunkCols;
            if (row0 < args.M && col < args.N) store_c(slice, col, row0);
            bulk_commit();                                            // also when nothing was stored: keeps the group count in step
          }
        }
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) {
          const uint32_t te = bar_tempty + 8 * part;
          mbar_arrive_cluster(CG == 1 ? te : mapa(te, 0));
        }
        }
      }
      if (ok && lane == 0 && args.trace && rank == 0 && warp == C::kEpi0) {
        args.trace[s].t_end = globaltimer();
        args.trace[s].epi_wait_acc = wait_epi;
      }
    }
    if (lane == 0) bulk_wait_all();   // every store of this warp has left shared memory and reached global memory
    __syncwarp();
    }
  }

  // ------------------------------------------------------------------ teardown
  tcgen05_fence_before();
  unit_sync<CG>();
  if (warp == 1) tmem_dealloc<CG>(tmem_base, kTmemCols);
  if (args.pinned && rank == 0 && threadIdx.x == 0) {
    // every unit took its rank at start-up; the last one to get here hands the counters back at zero, so the next
    // launch that is given this set needs no clearing in between (and keeps its place right behind this kernel)
    __threadfence();
    if (atomicAdd(args.die_count + 2, 1) == args.units - 1) {
      args.die_count[0] = 0; args.die_count[1] = 0; args.die_count[2] = 0; args.die_count[3] = 0; args.die_count[4] = 0;
      __threadfence();
    }
  }
  // An overlapped launch never waited for its predecessor; it must still not COMPLETE before it, or whatever follows
  // on the stream (a copy of the predecessor's C, an event) could run too early.  One thread holds the CTA's exit
  // until the predecessor grid has completed and its writes are visible; by now that is almost always the case.
  if (args.overlap && threadIdx.x == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Self-test of the bounded wait: a barrier nobody arrives on.  The wait must give up after
// `timeout_ns`, record its code and let the kernel end normally.
__global__ void selftest_wait_kernel(int32_t* status, unsigned long long timeout_ns, unsigned long long* waited_ns) {
  __shared__ __align__(8) unsigned long long bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const unsigned long long t0 = globaltimer();
    const bool ok = mbar_wait_slow(smem_u32(&bar), 0, status, (kRoleEpilogue << 8) | 0x7f, timeout_ns);
    *waited_ns = ok ? 0ull : globaltimer() - t0;
  }
}

int selftest_timeout(int32_t* status_dev, int timeout_us, int32_t* code_host, int64_t* waited_us_host) {
  unsigned long long* d_waited = nullptr;
  cudaError_t e = cudaMalloc(&d_waited, sizeof(unsigned long long));
  if (e == cudaSuccess) e = cudaMemset(status_dev, 0, sizeof(int32_t));
  if (e == cudaSuccess) {
    selftest_wait_kernel<<<1, 32>>>(status_dev, (unsigned long long)timeout_us * 1000ull, d_waited);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  unsigned long long waited = 0;
  int32_t code = 0;
  if (e == cudaSuccess) e = cudaMemcpy(&waited, d_waited, sizeof waited, cudaMemcpyDeviceToHost);
  if (e == cudaSuccess) e = cudaMemcpy(&code, status_dev, sizeof code, cudaMemcpyDeviceToHost);
  if (e == cudaSuccess) e = cudaMemset(status_dev, 0, sizeof(int32_t));
  cudaFree(d_waited);
  if (e != cudaSuccess) { set_error("wait self-test failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
  *code_host = code;
  *waited_us_host = (int64_t)(waited / 1000ull);
  return SP_OK;
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  });
  return fn;
}

// Row-major [rows, cols] matrix of 2-byte (bf16) or 4-byte (fp32) elements, box = box_rows x 128 bytes, 128-byte swizzle.
int make_map(CUtensorMap* m, const void* base, int64_t rows, int64_t cols, int box_rows, bool f32) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) { set_error("cuTensorMapEncodeTiled is not available from the driver"); return SP_ERR_CUDA; }
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * (f32 ? 4 : 2)};
  cuuint32_t box[2] = {f32 ? 32u : 64u, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled failed (CUresult %d)", (int)r); return SP_ERR_CUDA; }
  return SP_OK;
}

// Row-major [rows, cols] fp32 matrix, box = box_rows x box_cols elements, no shared-memory swizzle; parts of a box
// outside the matrix read as zero.
int make_map_plain(CUtensorMap* m, const void* base, int64_t rows, int64_t cols, int box_rows, int box_cols) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) { set_error("cuTensorMapEncodeTiled is not available from the driver"); return SP_ERR_CUDA; }
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled failed (CUresult %d)", (int)r); return SP_ERR_CUDA; }
  return SP_OK;
}

// Co-resident persistent units for one tile shape: one CTA per SM, or as many CTA pairs as the
// device can hold at once (asked of the occupancy calculator, cached per shape).
template <int CG, int BN>
static int max_units() {
  static int cached[64] = {};      // per device
  using C = Cfg<CG, BN>;
  auto kern = gemm_kernel<CG, BN, false, false, false>;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return -1;
  if (cached[dev & 63] > 0) return cached[dev & 63];
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
  int units = sms / CG;
  if (CG == 2) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::kSmemBytes) != cudaSuccess) return -1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(sms / CG * CG));
    cfg.blockDim = dim3(C::kThreads);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CG; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) == cudaSuccess && n > 0 && n < units) units = n;
    cudaGetLastError();
  }
  cached[dev & 63] = units;
  return units;
}

int gemm_units(int tile_m, int tile_n, int64_t T) {
  int64_t units = tile_m == 256 ? (tile_n == 128 ? max_units<2, 128>() : tile_n == 256 ? max_units<2, 256>() : max_units<2, 512>())
                                : (tile_n == 128 ? max_units<1, 128>() : max_units<1, 256>());
  if (units <= 0) return -1;
  if (units > T) units = T;
  return (int)units;
}

template <int CG, int BN, bool B_NK, bool OUT_F32, bool DYN>
static int launch_variant(const GemmCall& call, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC,
                          const GemmArgs& args) {
  using C = Cfg<CG, BN>;
  auto kern = gemm_kernel<CG, BN, B_NK, OUT_F32, DYN>;
  static uint64_t configured = 0;  // per instantiation, one bit per device
  cudaError_t e = cudaSuccess;
  if (first_use_on_this_device(configured)) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::kSmemBytes);
    if (e != cudaSuccess) { configured = 0; set_error("cudaFuncSetAttribute(smem=%u) failed: %s", C::kSmemBytes, cudaGetErrorString(e)); return SP_ERR_CUDA; }
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((args.clc ? args.sched.T : args.units) * CG));   // one cluster per tile, or per persistent unit
  cfg.blockDim = dim3(C::kThreads);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = call.stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CG;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  e = cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmC, args);
  if (e != cudaSuccess) { set_error("kernel launch failed: %s", cudaGetErrorString(e)); return SP_ERR_CUDA; }
  return SP_OK;
}

template <int CG, int BN, bool DYN>
static int launch_layout(const GemmCall& call, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC,
                         const GemmArgs& args) {
  if (call.b_nk) {
    return call.out_f32 ? launch_variant<CG, BN, true, true, DYN>(call, tmA, tmB, tmC, args)
                        : launch_variant<CG, BN, true, false, DYN>(call, tmA, tmB, tmC, args);
  }
  return call.out_f32 ? launch_variant<CG, BN, false, true, DYN>(call, tmA, tmB, tmC, args)
                      : launch_variant<CG, BN, false, false, DYN>(call, tmA, tmB, tmC, args);
}

template <int CG, int BN>
static int launch_shape(const GemmCall& call, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC,
                        const GemmArgs& args) {
  return (args.clc || args.steal) ? launch_layout<CG, BN, true>(call, tmA, tmB, tmC, args)
                                  : launch_layout<CG, BN, false>(call, tmA, tmB, tmC, args);
}

// Tensor maps of recent calls, per host thread: a map is a pure function of (address, extents, box, element type), so a
// call that repeats a matrix (the usual case: the same operands launch after launch) re-uses the encoded 128 bytes
// instead of asking the driver again.  Round-robin replacement.
struct MapKey {
  const void* base; int64_t rows, cols; int box_rows; int f32;
  bool operator==(const MapKey& o) const { return base == o.base && rows == o.rows && cols == o.cols && box_rows == o.box_rows && f32 == o.f32; }
};
static int cached_map(CUtensorMap* out, const void* base, int64_t rows, int64_t cols, int box_rows, bool f32) {
  constexpr int kEntries = 24;
  struct Entry { MapKey key; CUtensorMap map; };
  static thread_local Entry cache[kEntries];
  static thread_local int used = 0, next = 0;
  const MapKey key{base, rows, cols, box_rows, f32 ? 1 : 0};
  for (int i = 0; i < used; ++i)
    if (cache[i].key == key) { *out = cache[i].map; return SP_OK; }
  const int rc = make_map(out, base, rows, cols, box_rows, f32);
  if (rc != SP_OK) return rc;
  const int slot = used < kEntries ? used++ : (next = (next + 1) % kEntries);
  cache[slot].key = key; cache[slot].map = *out;
  return SP_OK;
}

static bool log_enabled() {
  static const bool on = getenv("SP_LOG") != nullptr;   // read once per process
  return on;
}

int launch_gemm(const GemmCall& call) {
  const int cg = call.tile_m / 128;
  const int bcols = (call.tile_n > 256 ? 256 : call.tile_n) / cg;  // B columns one CTA supplies to one MMA
  CUtensorMap tmA, tmB, tmC;
  int rc = cached_map(&tmC, call.C, call.M, call.N, 32, call.out_f32 != 0);   // one epilogue warp stores 32 rows x 128 bytes
  if (rc != SP_OK) return rc;
  rc = cached_map(&tmA, call.A, call.M, call.K, 128, false);
  if (rc != SP_OK) return rc;
  if (call.b_nk) rc = cached_map(&tmB, call.B, call.N, call.K, bcols, false);   // N x K, K contiguous: one box of bcols rows
  else rc = cached_map(&tmB, call.B, call.K, call.N, 64, false);                // K x N, N contiguous: boxes of 64 k x 64 n
  if (rc != SP_OK) return rc;

  GemmArgs args;
  args.C = call.C;
  args.perm = call.perm_dev;
  args.status = call.status_dev;
  args.trace = call.trace_dev;
  args.M = (int)call.M; args.N = (int)call.N; args.K = (int)call.K;
  args.kblocks = (int)((call.K + kBK - 1) / kBK);
  args.units = gemm_units(call.tile_m, call.tile_n, call.sched.T);
  if (args.units <= 0) { set_error("could not size the grid"); return SP_ERR_CUDA; }
  if (call.b_nk) {
    // K-major B: rows of 128 bytes, 8-row groups 1024 bytes apart; k advances inside the swizzle row
    args.b_lbo = 16; args.b_sbo = 1024; args.b_kstep = kUmmaK * 2;
  } else {
    // MN-major B: a box is 64 k-rows of 128 bytes (64 n); groups of 8 k-rows are 1024 bytes apart
    // (stride offset); the next 64 n live in the next box, 8192 bytes on (leading offset)
    args.b_lbo = 64 * kBK * 2; args.b_sbo = 1024; args.b_kstep = kUmmaK * 128;
  }
  args.steal = 0;
  args.pinned = 0; args.half0 = 0; args.units_on_die[0] = args.units_on_die[1] = 0; args.die_count = nullptr;
  for (int i = 0; i < 8; ++i) args.die_mask[i] = 0;
  if (call.pinned) {
    const int cg_ = call.tile_m / 128;
    args.pinned = 1;
    args.steal = call.steal;
    args.half0 = call.half0;
    args.units_on_die[0] = call.sms_on_die[0] / cg_;
    args.units_on_die[1] = call.sms_on_die[1] / cg_;
    args.die_count = call.die_count_dev;
    for (int i = 0; i < 8; ++i) args.die_mask[i] = call.die_mask[i];
    if (args.units != args.units_on_die[0] + args.units_on_die[1]) {
      set_error("die-pinned scheduling needs every SM to host one CTA (%d units launched, %d expected)", args.units,
                args.units_on_die[0] + args.units_on_die[1]);
      return SP_ERR_UNSUPPORTED;
    }
    // The tile space is cut into two equal halves, the SMs not always (72 / 76 has been measured): each half is
    // served by half of the units; the surplus units of the larger side take the top ranks of the other half
    // (the same rule that covers uneven placement), so both halves finish together.
    args.units_on_die[0] = (args.units + 1) / 2;
    args.units_on_die[1] = args.units / 2;
  }
  args.sched = call.sched;
  args.sk = SkPlan{0, args.units, call.sched.T};   // no tail: every slot is a whole tile
  args.sk_ws = nullptr; args.sk_flags = nullptr; args.sk_epoch = 0;
  args.overlap = call.overlap;
  args.clc = call.clc;
  args.k_alternate = call.k_alternate;
  args.hint_a = call.hint_a; args.hint_b = call.hint_b; args.hint_c = call.hint_c;
  if (call.stream_k) {
    // units are not capped by the tile count here: a problem smaller than a wave is spread over all of them
    const int all_units = gemm_units(call.tile_m, call.tile_n, kMaxTiles);
    const SkPlan plan = all_units > 0 ? sk_plan(call.sched.T, all_units, args.kblocks) : args.sk;
    if (plan.tiles > 0) {
      if ((size_t)all_units * call.tile_m * call.tile_n * sizeof(float) > kSkWorkspaceBytes ||
          (size_t)all_units * cg * 4 * sizeof(int32_t) > kSkFlagBytes) {
        set_error("stream-K workspace too small for %d units of %dx%d", all_units, call.tile_m, call.tile_n);
        return SP_ERR_UNSUPPORTED;
      }
      args.units = all_units;
      args.sk = plan;
      args.sk_ws = call.sk_ws_dev;
      args.sk_flags = call.sk_flags_dev;
      args.sk_epoch = call.sk_epoch;
    }
  }

  if (log_enabled()) {   // diagnostics on request: which variant runs, and how
    const int stages = cg == 1 ? (call.tile_n == 128 ? Cfg<1, 128>::kStages : Cfg<1, 256>::kStages)
                               : (call.tile_n == 128 ? Cfg<2, 128>::kStages : call.tile_n == 256 ? Cfg<2, 256>::kStages : Cfg<2, 512>::kStages);
    fprintf(stderr, "[swizzleperf] gemm %dx%dx%d tile %dx%d (%d CTA%s per tile) scheme %d T=%d units=%d grid=%d stages=%d kblocks=%d "
                    "b=%s out=%s table=%d pinned=%d split_tail=%d/%d clc=%d overlap=%d k_alternate=%d steal=%d\n",
            args.M, args.N, args.K, call.tile_m, call.tile_n, cg, cg > 1 ? "s" : "", call.sched.scheme, call.sched.T, args.units,
            (args.clc ? call.sched.T : args.units) * cg, stages, args.kblocks, call.b_nk ? "NxK" : "KxN", call.out_f32 ? "fp32" : "bf16",
            call.sched.use_table, args.pinned, args.sk.tiles, args.sk.units, args.clc, args.overlap, args.k_alternate, args.steal);
  }
  if (cg == 1) return call.tile_n == 128 ? launch_shape<1, 128>(call, tmA, tmB, tmC, args) : launch_shape<1, 256>(call, tmA, tmB, tmC, args);
  if (call.tile_n == 512) return launch_shape<2, 512>(call, tmA, tmB, tmC, args);
  return call.tile_n == 128 ? launch_shape<2, 128>(call, tmA, tmB, tmC, args) : launch_shape<2, 256>(call, tmA, tmB, tmC, args);
}

}  // namespace sp
