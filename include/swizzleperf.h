/* swizzleperf.h -- C ABI of libswizzleperf.so
 *
 * A tiled dense bf16 GEMM for NVIDIA B200 (sm_100a) whose block-to-output-tile mapping
 * is a programmable "swizzle": a bijective remap of tile ids, as in the GEMM case study
 * of the SwizzlePerf paper (arXiv 2508.20258, appendix "Case Study: GEMM Swizzling").
 * Two memory-bound workloads of the paper's suite, a tiled transpose and a 2-D stencil, run
 * under the same remaps (sp_transpose, sp_stencil2d).
 *
 * Vocabulary.  C (M x N) = A (M x K) . B (K x N) is cut into Tm x Tn output tiles,
 * Tm = ceil(M / tileM), Tn = ceil(N / tileN), T = Tm * Tn.  The logical id of tile
 * (tm, tn) is t = tm * Tn + tn (the row-major decomposition pid_m = pid / Tn,
 * pid_n = pid % Tn of the paper's hardware-unaware listing).  Blocks are issued in
 * slot order s = 0 .. T-1; the remap is perm[s] = t, "the block issued at slot s
 * computes tile t" -- the direction of the paper's  pid = f(pid)  (hardware id in,
 * logical id out).  A remap must be a bijection on [0, T); the paper counts anything
 * else as a broken mapping, and every entry point here rejects it before any launch.
 *
 * Conventions.  Every function returns an sp_status (0 = success) and never throws,
 * aborts or prints.  "host" / "device" below says where a pointer must point.  The
 * caller owns every buffer it passes; the library owns only its internal caches (tile
 * tables, a status word with scheduling counters, staging for the host entry point, the
 * workspace of SP_FLAG_STREAM_K), released by sp_shutdown().  All device work is enqueued on the
 * caller's stream; nothing synchronises unless stated.
 */
#ifndef SWIZZLEPERF_H_
#define SWIZZLEPERF_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SP_OK = 0,
  SP_ERR_INVALID_ARG = 1,   /* NULL pointer, non-positive size, bad parameter value            */
  SP_ERR_NOT_BIJECTIVE = 2, /* the requested remap does not hit every tile id exactly once     */
  SP_ERR_UNSUPPORTED = 3,   /* tile shape / dtype / size outside what the kernels implement    */
  SP_ERR_ALIGNMENT = 4,     /* pointer not 16-byte aligned, or K / N not a multiple of 8       */
  SP_ERR_CUDA = 5,          /* a CUDA runtime or driver call failed (see sp_last_error)        */
  SP_ERR_TIMEOUT = 6,       /* a bounded device-side wait expired; output is undefined         */
  SP_ERR_DEVICE = 7         /* no usable sm_100 device                                         */
} sp_status;

/* Tile orders.  SP_XCD is the paper's formula; the others are this library's. */
typedef enum {
  SP_ROW_MAJOR = 0, /* perm[s] = s (the paper's unswizzled baseline)                                        */
  SP_COL_MAJOR = 1, /* tile columns outer, tile rows inner                                                  */
  SP_GROUP_M = 2,   /* supertiles of `group` tile rows: per band walk columns, per column walk band rows    */
  SP_GROUP_N = 3,   /* supertiles of `group` tile columns (transpose of SP_GROUP_M)                         */
  SP_MORTON = 4,    /* Z-order on the enclosing 2^k square (k minimal), cells outside the grid skipped;     */
                    /*   the longer grid side is walked by the curve's y (odd bits)                         */
  SP_HILBERT = 5,   /* Hilbert order on the same square, same skipping, curve from (0,0) to (2^k-1,0)       */
  SP_XCD = 6,       /* paper, GEMM listing: within each window of `wave` slots of size n,                   */
                    /*   p -> (p % X) * ceil(n / X) + p / X, X = num_xcds.  With xcd_balanced = 1 the       */
                    /*   remainder-aware form p -> (p % X) * (n / X) + min(p % X, n % X) + p / X, which is  */
                    /*   a bijection for every n and equals the printed form when X divides n.              */
  SP_DIE_SPLIT = 7, /* tile space cut in two halves along split_axis (half 0 gets the ceil), each half a    */
                    /*   grid of its own ordered by inner_scheme; perm = half 0 then half 1, or alternating */
                    /*   (slot parity = half, the paper's formula with two chiplets) when interleave = 1    */
  SP_CUSTOM = 8,    /* caller-supplied table                                                                */
  SP_HILBERT_RECT = 9 /* generalised Hilbert curve laid directly over the Tm x Tn rectangle (the published         */
                    /*   construction for arbitrary rectangles): no cell outside the grid is visited, consecutive   */
                    /*   slots are adjacent tiles (at most one diagonal step); on 2^k squares it is a Hilbert curve. */
                    /*   Not in the paper.  Not available as inner order of SP_DIE_SPLIT.                            */
} sp_scheme;

/* sp_params.flags */
#define SP_FLAG_TRACE 1u      /* reserved for sp_gemm_trace */
#define SP_FLAG_SERPENTINE 4u /* SP_GROUP_M / SP_GROUP_N (also as inner order of SP_DIE_SPLIT), in sp_tile_map* and sp_gemm*:
                                 odd bands are walked in the opposite direction, so a band starts on the panels the
                                 previous band used last */
#define SP_FLAG_DIE_PINNED 2u /* sp_gemm* with SP_DIE_SPLIT, interleave = 0: the persistent units whose SM sits on L2 half d
                                 (measured by the topology probe, cached) run only the slots of half d of the tile space,
                                 in arrival order on that half.  Needs at least as many tiles as SMs / CTAs-per-tile;
                                 SP_ERR_UNSUPPORTED if the probe finds no usable two-way structure.  The output is the same, and every
                                 tile runs exactly once wherever the units land.  At most 64 such launches in flight per device. */

#define SP_FLAG_STREAM_K 8u   /* sp_gemm / sp_gemm_trace / sp_gemm_host, tiles up to 256x256: wave quantisation.  The paper's
                                 remap picks the tile of a slot and has no counterpart for this.  When the persistent units U
                                 do not divide the tile count T, the last R = T mod U slots of the order are split along k:
                                 each of their tiles goes to f = min(U / R, kblocks / 4, 8) units, piece i taking k-blocks
                                 [i * kblocks / f, (i + 1) * kblocks / f) (sp_streamk_plan lists the pieces); nothing is
                                 split when f < 2.  Pieces with the same i walk k in step, so they still share operand
                                 panels in L2.  A unit whose piece ends before the tile's last k-block writes an fp32 partial
                                 to a library workspace; the unit with the last piece adds the partials (fixed order) and
                                 stores the tile.  C is then the same sum taken in a different order: equal run to run for
                                 one (shape, tile, unit count), no longer bit-identical across orders or to a launch without
                                 the flag.  Device waits on partials are bounded like every other wait and only ever point
                                 to lower block indices.  The workspace (about 19 MB) is allocated on first use per stream,
                                 at most 8 streams per device; not available in sp_gemm_noalloc or with SP_FLAG_DIE_PINNED
                                 (SP_ERR_INVALID_ARG) nor for the 256x512 tile (SP_ERR_UNSUPPORTED).  In a trace the record
                                 of a split tile describes the piece that stored it. */

#define SP_FLAG_CLC 32u       /* sp_gemm / sp_gemm_trace / sp_gemm_host: dynamic scheduling by cluster launch control.  The grid has
                                 one cluster per tile instead of one per persistent unit; the clusters that get to run compute
                                 the slot of their own index and then keep asking the hardware to cancel a cluster that has not
                                 started yet and to hand them its index (clusterlaunchcontrol.try_cancel), until none is left.
                                 Slots are then taken in the order the hardware starts and cancels clusters, first come first
                                 served, not with a fixed stride; every tile still runs exactly once and C has the same bits.
                                 The counterpart, on this hardware, of the paper's premise that the scheduler hands out
                                 consecutive block ids in a fixed pattern.  Not with SP_FLAG_DIE_PINNED or SP_FLAG_STREAM_K
                                 (SP_ERR_INVALID_ARG). */
#define SP_FLAG_OVERLAP 16u   /* sp_gemm only.  The caller states that this launch is independent of the kernel before it on the
                                 stream: it reads nothing that kernel writes, and it may start writing C while that kernel is
                                 still running.  Every GEMM launch of this library is made with programmatic stream
                                 serialisation and signals at its start that its successor may be scheduled; an ordinary
                                 launch then waits, after its set-up and before it touches global memory, until the kernel
                                 before it has completed and its writes are visible (so only launch latency and set-up
                                 overlap, and the stream order is the usual one); a launch with this flag does not wait.  CTAs of the next GEMM then take over SMs as the CTAs of the
                                 previous one finish, which fills the partly empty last wave of back-to-back independent
                                 GEMMs.  The paper has no counterpart.  Not with SP_FLAG_DIE_PINNED,
                                 SP_FLAG_STREAM_K or tracing (SP_ERR_INVALID_ARG).  It still completes after its predecessor, so the
                                 stream order seen by everything else (copies, events, other kernels) is unchanged. */

#define SP_FLAG_STEAL 4096u   /* sp_gemm / sp_gemm_trace / sp_gemm_host, together with SP_FLAG_DIE_PINNED.  The slots of each half
                                 of the tile space are handed out by ticket (one atomic per tile) to the units of that L2
                                 half, in slot order; a unit that finds its own half's queue empty takes tickets of the other
                                 half, so no unit idles while a tile is still waiting.  Without the flag each unit owns a
                                 fixed stride of its half and a half that finishes early waits for the other.  Matters when
                                 the halves hold unequal work (an odd number of tile rows, a ragged edge) or the GPU is
                                 shared.  C has the same bits either way (every tile is computed whole, by one unit).  No
                                 counterpart in the paper, whose blocks cannot trade work once launched. */
#define SP_FLAG_K_ALTERNATE 64u /* sp_gemm* only.  Every other tile a persistent unit works on walks the K dimension from the
                                 far end (k-blocks in descending order).  The tiles of one round advance through K in step, so
                                 what L2 holds when a round ends is the end of the K range of that round's operand panels; a
                                 round that shares panels with it and starts there finds them still cached, where a round
                                 that starts over at k = 0 finds them evicted: fewer DRAM reads (a fifth fewer at 8192^3 under
                                 bands of eight) and, at the power limit, less time.  The paper has no counterpart: its remap
                                 chooses which tile a block computes, never the order inside a tile.  C = A.B as before, but
                                 the fp32 sum of a tile is taken in the order its k-blocks arrive, so the rounding of C
                                 depends on which round a tile ran in, hence on the order and the unit count (like
                                 SP_FLAG_STREAM_K, and within the same tolerance); with exactly representable partial sums
                                 (small integers) C has the same bits either way.  Combines with every scheme and flag. */

/* sp_gemm* only.  L2 eviction priorities for the lines a GEMM's bulk copies bring in or write (the
 * paper has no counterpart: its lever is which block runs where, not what the cache keeps).  evict_first marks lines as
 * the first to go when room is needed (an operand that is streamed once per band, C tiles that are written and never
 * read), evict_last as lines to keep (the operand panels a band of tiles shares from round to round).  Results are
 * unchanged; only the cache's replacement choices are.  A and B may each be given at most one of the two. */
#define SP_FLAG_HINT_C_EVICT_FIRST 128u
#define SP_FLAG_HINT_A_EVICT_FIRST 256u
#define SP_FLAG_HINT_B_EVICT_FIRST 512u
#define SP_FLAG_HINT_A_EVICT_LAST 1024u
#define SP_FLAG_HINT_B_EVICT_LAST 2048u

typedef struct {
  uint32_t struct_size;       /* must be sizeof(sp_params)                                                  */
  int32_t group;              /* G >= 1 for SP_GROUP_M / SP_GROUP_N                                         */
  int32_t num_xcds;           /* X >= 1 for SP_XCD                                                          */
  int32_t wave;               /* W for SP_XCD: window length in slots; 0 means W = T                        */
  int32_t xcd_balanced;       /* SP_XCD: 0 = formula exactly as printed (may be rejected), 1 = balanced     */
  int32_t split_axis;         /* SP_DIE_SPLIT: 0 = halve the tile rows, 1 = halve the tile columns          */
  int32_t inner_scheme;       /* SP_DIE_SPLIT: order inside each half: SP_ROW_MAJOR .. SP_HILBERT           */
  int32_t inner_group;        /* SP_DIE_SPLIT: G of the inner scheme                                        */
  int32_t interleave;         /* SP_DIE_SPLIT: 0 = concatenated halves, 1 = alternating merge               */
  const int32_t* custom_perm; /* SP_CUSTOM: HOST array of T tile ids (validated, copied)                    */
  int32_t tile_m, tile_n;     /* sp_gemm*: 128x128, 128x256 (one CTA per tile), 256x128, 256x256 (a CTA pair */
                              /*   per tile) or 256x512 (a CTA pair runs two 256x256 MMA tiles that share    */
                              /*   the A panel); 0,0 = 256x256.  Ignored by sp_tile_map*.                    */
  int32_t out_dtype;          /* sp_gemm*: 0 = C is bf16 (round to nearest even), 1 = C is fp32             */
  int32_t b_layout;           /* sp_gemm*: 0 = B is K x N row-major, 1 = B is N x K row-major               */
  uint32_t flags;             /* 0, or any of SP_FLAG_DIE_PINNED, _SERPENTINE, _STREAM_K, _OVERLAP, _CLC, _K_ALTERNATE, _STEAL, _HINT_* */
} sp_params;

/* One record per tile, written by sp_gemm_trace. */
typedef struct {
  int32_t slot;      /* issue slot s                                   */
  int32_t tile;      /* logical tile id executed at that slot          */
  int32_t smid;      /* %smid of the (leader) CTA that ran it          */
  int32_t unit;      /* index of the persistent CTA / CTA pair         */
  uint64_t t_begin;  /* %globaltimer (ns) when its first load was issued                      */
  uint64_t t_end;    /* %globaltimer when its last store was issued                            */
  uint64_t t_mma_begin;   /* %globaltimer when the MMA issuer started on the tile               */
  uint64_t t_mma_issued;  /* %globaltimer when it had issued the tile's last MMA                */
  uint32_t mma_wait_data; /* SM cycles the MMA issuer waited for operand stages of this tile    */
  uint32_t mma_wait_acc;  /* SM cycles it waited for a free accumulator buffer                  */
  uint32_t load_wait_stage; /* SM cycles the producer waited for a free stage                   */
  uint32_t epi_wait_acc;  /* SM cycles the first epilogue warp waited for the accumulator       */
} sp_trace_rec;

/* Number of tiles T = ceil(M/tileM) * ceil(N/tileN); -1 on non-positive arguments. */
int64_t sp_tile_count(int64_t M, int64_t N, int32_t tileM, int32_t tileN);

/* The remap (paper: the recomputed pid of each block).
 *   out_perm : HOST, caller-owned, T int32 entries; out_perm[s] = tile run at slot s.
 *   params   : HOST; may be NULL for schemes that need no parameter.
 * Errors: SP_ERR_INVALID_ARG (sizes <= 0, T > 2^24, G < 1, X < 1, wave < 0, bad axis / inner scheme,
 * wrong struct_size, NULL out_perm), SP_ERR_NOT_BIJECTIVE (printed SP_XCD form when X does not
 * divide a window, bad custom table).  On any error out_perm is left untouched.  Pure host code. */
int sp_tile_map(int64_t M, int64_t N, int32_t tileM, int32_t tileN, int scheme, const sp_params* params,
                int32_t* out_perm);

/* Same remap, evaluated by the DEVICE code the GEMM scheduler uses, written to
 *   out_perm_dev : DEVICE, T int32 entries, on `stream` (asynchronous).
 * Validation (including bijectivity) happens on the host first; same error codes. */
int sp_tile_map_device(int64_t M, int64_t N, int32_t tileM, int32_t tileN, int scheme, const sp_params* params,
                       int32_t* out_perm_dev, void* stream);

/* C = A . B under the given tile order (paper: the GEMM whose block ids are remapped).
 *   A : DEVICE, bf16, M x K row-major, read-only.
 *   B : DEVICE, bf16, K x N row-major (b_layout 0) or N x K row-major (b_layout 1), read-only.
 *   C : DEVICE, M x N row-major, bf16 or fp32 per params->out_dtype; fully overwritten; must not alias A or B.
 *   stream : cudaStream_t (NULL = default stream).  Asynchronous.
 * Products are accumulated in fp32 on the tensor cores.  M and N need not be tile multiples.
 * Errors (all detected on the host, nothing launched): as sp_tile_map, plus SP_ERR_ALIGNMENT (A, B or C not
 * 16-byte aligned; K or N not a multiple of 8), SP_ERR_UNSUPPORTED (tile shape), SP_ERR_DEVICE, SP_ERR_CUDA.
 * The first call for a given (grid, scheme) may allocate a cached tile table, fills it on `stream` and synchronises
 * `stream` once before the table becomes visible to other calls (so a call on any other stream or host thread that
 * finds it may launch at once); later calls allocate nothing, synchronise nothing and
 * issue only the kernel launch (tensor maps of recently used matrices are kept per host thread), so after one warm-up call per
 * (shape, scheme, params) further calls can be recorded into a CUDA graph by stream capture and replayed; the
 * pointers and the order are then those of the recording.
 * A device-side wait that expires is reported by sp_get_status, not here.
 * With the environment variable SP_LOG set when the library is first used, every launch writes one line to stderr (shape, tile, variant, grid, pipeline
 * depth, flags in effect); nothing is ever written to stdout. */
int sp_gemm(const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t K, int scheme,
            const sp_params* params, void* stream);

/* sp_gemm that also records, for every tile, where and when it ran.
 *   trace_dev : DEVICE, T sp_trace_rec entries, indexed by slot. */
int sp_gemm_trace(const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t K, int scheme,
                  const sp_params* params, void* stream, sp_trace_rec* trace_dev);

/* sp_gemm for callers whose matrices live in HOST memory (pinned or pageable), same layouts and dtypes:
 * copies A and B to a device staging area owned by the library (grown on demand, kept until sp_shutdown),
 * runs sp_gemm, copies C back, and synchronises `stream`; C_host is valid on return.  With 4096 rows or more (and
 * no caller table) M is split into row blocks (256 rows, more when M exceeds 8192: C trails A by one block, so
 * small blocks leave little to do once the last byte of A has arrived), each computed
 * by its own sp_gemm under the same scheme applied to the block's tile grid, so that copies in both directions overlap
 * the compute; the result is the same (a die-pinned order is applied unpinned to a row block with fewer tiles than
 * the device has persistent units).  The staging area is shared: calls from several host threads are served one after
 * the other (the function holds a lock for its whole duration).  Adds SP_ERR_TIMEOUT
 * to sp_gemm's errors. */
int sp_gemm_host(const void* A_host, const void* B_host, void* C_host, int64_t M, int64_t N, int64_t K, int scheme,
                 const sp_params* params, void* stream);

/* sp_gemm for callers that must not allocate device memory.  (The paper has no counterpart: this is a
 * deployment variant of sp_gemm, same arguments, same result.)
 *
 * Who needs it: a process that has given the whole GPU to its own memory pool, where a cudaMalloc made by a
 * library fails or is charged to a budget nobody planned for; and latency-critical loops, where the
 * device-wide synchronisation hidden in cudaMalloc / cudaFree is unacceptable.  sp_gemm allocates (once, cached)
 * a tile table for non-arithmetic orders and a status word; here both live in a fixed array inside the
 * library image, so this call performs no cudaMalloc, cudaFree or other allocating call.
 *
 *   A, B, C, M, N, K, scheme, params, stream : as sp_gemm (DEVICE buffers owned by the caller), except that of the
 *                 flags only SP_FLAG_SERPENTINE, SP_FLAG_K_ALTERNATE and SP_FLAG_HINT_* are accepted: SP_FLAG_DIE_PINNED and SP_FLAG_STREAM_K need memory that
 *                 sp_gemm allocates, SP_FLAG_OVERLAP and SP_FLAG_CLC launches could run beside their predecessor and
 *                 find the shared array rewritten under them (each returns SP_ERR_INVALID_ARG here).
 *   status_host : HOST, may be NULL.  NULL: the call is asynchronous and an expired device-side wait goes
 *                 unreported.  Non-NULL: the call synchronises `stream`, stores the raw status word there and
 *                 returns SP_ERR_TIMEOUT if it is non-zero.
 * Limits and sharing:
 *   - at most 65536 tiles (ceil(M/tile_m) * ceil(N/tile_n)); more returns SP_ERR_UNSUPPORTED.  The array
 *     (about 257 KiB) is held by every GPU context that loads the library until the process exits.
 *   - every call on a device uses the same array, and the array keeps the previous call's contents: each call
 *     clears the status word and, unless the array already holds exactly the table it needs (same grid, order and
 *     parameters, or the same caller table, as the call before), rewrites the table, on `stream`, before its kernel.
 *     Two calls that overlap on the GPU (different streams, or several host threads) race on it; serialise them.
 *   - a new SP_CUSTOM table is uploaded from pageable host memory: that call synchronises `stream` once, whatever
 *     status_host is; repeating the same table does not.
 *   - the first call on each device looks up the array's device address (with that device current);
 *     make that first call outside any stream capture.
 * Errors: as sp_gemm, plus SP_ERR_UNSUPPORTED for too many tiles. */
int sp_gemm_noalloc(const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t K, int scheme,
                    const sp_params* params, void* stream, int32_t* status_host);

/* out (N x M) = transpose of in (M x N) for 16-bit elements, under a tile order (paper: the transpose kernel, its
 * largest reported win, whose tile grid is re-ordered for L2 locality of both the reads and the transposed writes).
 * The matrix is cut into SP_TRANSPOSE_TILE x SP_TRANSPOSE_TILE tiles; `scheme` / `params` order that tile grid exactly
 * as for sp_tile_map(M, N, 64, 64, ...); persistent CTAs take slots with a fixed stride.
 *   in  : DEVICE, M x N row-major, 2-byte elements (bf16, fp16, int16: bits are moved, not interpreted), read-only.
 *   out : DEVICE, N x M row-major, fully overwritten; must not overlap `in`.
 * Errors: SP_ERR_INVALID_ARG, SP_ERR_ALIGNMENT (pointers not 16-byte aligned, M or N not a multiple of 8),
 * SP_ERR_NOT_BIJECTIVE, SP_ERR_UNSUPPORTED, SP_ERR_DEVICE, SP_ERR_CUDA.  Asynchronous on `stream`. */
#define SP_TRANSPOSE_TILE 64
int sp_transpose(const void* in, void* out, int64_t M, int64_t N, int scheme, const sp_params* params, void* stream);

/* One sweep of the five-point stencil over an fp32 grid, under a tile order (paper: "Stencil 2D", one of its science
 * kernels, whose block grid is re-ordered so that blocks sharing halo data meet in one L2; the paper does not print
 * the stencil: the five-point star with the rim carried over is this library's reading):
 *   out[i][j] = c_center * in[i][j] + c_neighbor * (in[i-1][j] + in[i+1][j] + in[i][j-1] + in[i][j+1])
 *                                                            for 0 < i < M-1 and 0 < j < N-1,
 *   out[i][j] = in[i][j]                                     on the rim (also the whole grid when M < 3 or N < 3).
 * Arithmetic in fp32: the four neighbours are added in pairs, (north + south) + (west + east), then one fused
 * multiply-add onto c_center * in[i][j].  The grid is cut into SP_STENCIL_TILE_M x SP_STENCIL_TILE_N tiles;
 * `scheme` / `params` order that tile grid exactly as for sp_tile_map(M, N, 64, 128, ...); persistent CTAs take
 * slots with a fixed stride.
 *   in  : DEVICE, M x N row-major fp32, read-only.
 *   out : DEVICE, M x N row-major fp32, fully overwritten; must not overlap `in`.
 * Errors: SP_ERR_INVALID_ARG (NULL, sizes, in == out, NaN coefficient), SP_ERR_ALIGNMENT (pointers not 16-byte
 * aligned, N not a multiple of 4), SP_ERR_NOT_BIJECTIVE, SP_ERR_UNSUPPORTED, SP_ERR_DEVICE, SP_ERR_CUDA.
 * Asynchronous on `stream`. */
#define SP_STENCIL_TILE_M 64
#define SP_STENCIL_TILE_N 128
int sp_stencil2d(const void* in, void* out, int64_t M, int64_t N, float c_center, float c_neighbor, int scheme,
                 const sp_params* params, void* stream);

/* Row softmax of an fp32 matrix, out[i][j] = exp(in[i][j] - max_j in[i][:]) / sum_j exp(in[i][j] - max_j in[i][:]), in
 * the two forms the paper's softmax case study contrasts (there the rows are reduced in two phases, the maximum first, then
 * the exponentials and their sum, with the chunks of a row spread over blocks; the remap the paper finds keeps a row's
 * chunks in one chiplet's L2 between the phases):
 *   mode SP_SOFTMAX_SINGLE_PASS        : blocks of whole rows pass through shared memory once; every byte crosses HBM
 *                                        once per direction.  A row of more than 16384 elements (one 64 KiB buffer) is
 *                                        shared by the ceil(N / 16384) CTAs (2 to 8; 8 instead of 7) of a thread-block cluster, which
 *                                        exchange their partial maxima and sums through distributed shared memory (faster
 *                                        than the two-phase form up to about 65536 elements per row, slower beyond: the
 *                                        more CTAs wait for each other per row, the more their skew costs); N <= 131072,
 *                                        else SP_ERR_UNSUPPORTED.  `scheme` / `params` order the row blocks, as for
 *                                        sp_tile_map(M, N, rows, N, ...) with, in integer arithmetic, rows =
 *                                        max(1, 12288 / N) for N > 1792 (blocks of at most 48 KiB, or one row; several warps on a
 *                                        row) and rows = min(96, max(8, 12288 / N / 8 * 8)) for N <= 1792 (a warp per row).
 *   mode SP_SOFTMAX_TWO_PHASE          : the matrix is cut into SP_SOFTMAX_TILE_M x SP_SOFTMAX_TILE_N tiles, ordered exactly as
 *                                        for sp_tile_map(M, N, 32, 512, ...).  A first launch leaves per tile and row
 *                                        the partial maximum and partial sum; a second one combines them per row, reads
 *                                        the tiles again (from L2 where they still are) and writes the result.
 *   mode SP_SOFTMAX_TWO_PHASE_REVERSED : the same, the second launch walking the slots backwards, so that it starts with
 *                                        the tiles the first one touched last.
 * Arithmetic in fp32; exp through the hardware's 2^x of (difference x log2 e); sums by lanes, then by shuffles.
 *   in  : DEVICE, M x N row-major fp32, finite values, read-only.
 *   out : DEVICE, M x N row-major fp32, fully overwritten; must not overlap `in`.
 * The two-phase modes keep their partials (8 bytes per row and column chunk) in device memory owned by the library,
 * grown on demand and shared by all calls on the device: two-phase calls that overlap on the GPU (different streams)
 * race on it; serialise them.
 * Errors: SP_ERR_INVALID_ARG (NULL, sizes, in == out, mode), SP_ERR_ALIGNMENT (pointers not 16-byte aligned, N not a
 * multiple of 4), SP_ERR_NOT_BIJECTIVE, SP_ERR_UNSUPPORTED, SP_ERR_DEVICE, SP_ERR_CUDA.  Asynchronous on `stream`. */
#define SP_SOFTMAX_TILE_M 32
#define SP_SOFTMAX_TILE_N 512
#define SP_SOFTMAX_SINGLE_PASS 0
#define SP_SOFTMAX_TWO_PHASE 1
#define SP_SOFTMAX_TWO_PHASE_REVERSED 2
int sp_softmax(const void* in, void* out, int64_t M, int64_t N, int32_t mode, int scheme, const sp_params* params,
               void* stream);

/* A starting configuration for sp_gemm on this hardware: tile shape, order and its parameters for a given problem.
 * The paper arrives at a remap by searching with measurements in the loop; this is the short table that this
 * library's own sweeps on B200 distil to (no counterpart in the paper, and no substitute for measuring: the search
 * loop of the Python package does that).  Rule: among the supported tiles, the one with the least estimated time
 * waves x tile area / (CTAs per tile x relative efficiency of the tile shape), waves = ceil(T / units), units = what
 * sp_gemm_units reports on the current device, or, with no device present, 74 CTA pairs / 148 CTAs; row-major when A and B together are at most 64 MiB (they stay in L2) or the tile grid is at most
 * ten tiles wide, column-major when it is at most ten tiles tall (both with SP_FLAG_K_ALTERNATE and
 * SP_FLAG_HINT_C_EVICT_FIRST when A and B together exceed 64 MiB), else bands of 8 tile columns (256x512 tile) or 8
 * tile rows (other tiles), walked serpentine-wise with SP_FLAG_K_ALTERNATE and SP_FLAG_HINT_C_EVICT_FIRST (the rounding
 * of C then depends on the order, within the usual tolerance); SP_FLAG_STREAM_K is set when the tiles fill at most half of the units and K is at least
 * 2048 (C then differs in rounding order from a launch without the flag).  Host code; no GPU needed.
 *   params : HOST, receives a complete sp_params (struct_size, tile_m, tile_n, group, out_dtype, b_layout set; the
 *            rest zero).   scheme : HOST, receives the sp_scheme.
 * Errors: SP_ERR_INVALID_ARG (NULL, sizes <= 0, bad out_dtype / b_layout). */
int sp_recommend(int64_t M, int64_t N, int64_t K, int32_t out_dtype, int32_t b_layout, sp_params* params, int* scheme);

/* Number of persistent CTAs (tile 128xN) or CTA pairs (tile 256xN) sp_gemm launches for T tiles;
 * slot s is run by unit s % units in round s / units.  Returns -1 on error. */
int sp_gemm_units(int32_t tile_m, int32_t tile_n, int64_t T);

/* The k-split of SP_FLAG_STREAM_K for T tiles of kblocks k-blocks (of 64) on `units` persistent units; host only, no
 * GPU needed.  The paper has no counterpart (see the flag).  Writes, for every unit u in [0, units), up to
 * SP_STREAMK_MAX_SEGMENTS segments in the order the unit walks them, as 4 int32 each at
 * out_segments[(u * SP_STREAMK_MAX_SEGMENTS + j) * 4]: {slot, k_begin, k_end, kind} with kind 0 = whole tile,
 * 1 = contributor (partial to the workspace), 2 = owner (adds the contributors' partials, stores); unused entries
 * have slot = -1 (with the present policy a unit has at most one segment).  *first_slot receives the first slot of
 * the split tail (T when nothing is split): slots below it are dealt out whole, slot s to unit s % units.
 * Returns SP_OK or SP_ERR_INVALID_ARG. */
#define SP_STREAMK_MAX_SEGMENTS 8
int sp_streamk_plan(int64_t T, int32_t units, int32_t kblocks, int32_t* first_slot, int32_t* out_segments);

/* Launch-order probe (the counterpart of the paper's "default scheduling policy" context):
 * launches `n_blocks` trivial blocks in clusters of `cluster` (1 or 2) and records for block b
 *   smid_host[b] = %smid, start_host[b] = %globaltimer at entry.  HOST arrays of n_blocks. Synchronous. */
int sp_probe_dispatch(int32_t n_blocks, int32_t cluster, int32_t* smid_host, uint64_t* start_host);

/* Topology probe (counterpart of the paper's parsed hardware context: number of XCDs, their L2s).
 * Every SM in turn times first-touch loads of the same SP_PROBE_LINES cache lines, each rewritten before the
 * round; SMs whose fast/slow pattern over the lines agrees share an L2 half (die).
 *   sm_to_die_host : HOST, capacity >= 1024 int32; entry [smid] = 0 or 1 (group 0 contains the lowest measured SM),
 *                    -1 if that SM could not be measured.
 *   n_sm           : HOST, receives the SM count.
 *   confidence     : HOST, mean |agreement| in [0,1]; near 0 means no measurable two-way structure.
 *   lat_host       : HOST, may be NULL; else n_sm * SP_PROBE_LINES uint32 minimum latencies in SM cycles.
 * Synchronous; allocates and frees its own buffers; takes a fraction of a second. */
#define SP_PROBE_LINES 128
int sp_probe_topology(int32_t* sm_to_die_host, int32_t* n_sm, float* confidence, uint32_t* lat_host);

/* Effective L2 capacity probe (counterpart of the paper's "L2 size per XCD" context).  For each working-set size every
 * participating SM reads the whole set repeatedly with loads that bypass L1; the aggregate read rate of the repeat passes
 * drops once the set no longer fits in what the L2 holds for those readers.
 *   sizes_bytes : HOST, n_sizes (1..256) working-set sizes, each a multiple of 16 in [4 KiB, 1 GiB].
 *   half        : -1 = all SMs read; 0 / 1 = only the SMs measured on that L2 half (runs the topology probe if needed).
 *   gbps_out    : HOST, n_sizes aggregate read rates in GB/s.
 * Synchronous; allocates and frees a buffer of the largest size. */
int sp_probe_l2_capacity(int32_t n_sizes, const int64_t* sizes_bytes, int32_t half, float* gbps_out);

/* Self-test (host only) of the rank assignment of die-pinned scheduling: with n0 / n1 units expected on the two L2
 * halves and arrivals0 of the n0 + n1 units actually landing on half 0, every (half, rank) pair must be handed out
 * exactly once.  Returns SP_OK, or SP_ERR_NOT_BIJECTIVE if the assignment would skip or repeat work. */
int sp_selftest_pinned_tickets(int32_t n0, int32_t n1, int32_t arrivals0);

/* Self-test of the bounded device-side wait every kernel role uses: a one-thread kernel waits on a barrier that
 * nothing arrives on, with a limit of timeout_us (1 .. 1000000).  The wait must expire, record its code and let the
 * kernel end normally (no trap, no fault; the context stays usable).
 *   code      : HOST, receives the status word the wait recorded (non-zero when it expired as designed).
 *   waited_us : HOST, receives how long the wait lasted.
 * Synchronous; clears the status word afterwards. */
int sp_selftest_timeout(int32_t timeout_us, int32_t* code, int64_t* waited_us);

/* Synchronises `stream`, then returns and clears the device status word of the current device:
 * SP_OK, or SP_ERR_TIMEOUT if a kernel gave up on a bounded wait since the last call.
 * *detail (HOST, may be NULL) receives the raw word (which wait, which role). */
int sp_get_status(void* stream, int32_t* detail);

/* Text for the last error on the calling thread; valid until that thread's next call. Never NULL. */
const char* sp_last_error(void);

/* Frees the library's caches on every device it touched.  No call may be in flight. */
void sp_shutdown(void);

#ifdef __cplusplus
}
#endif
#endif /* SWIZZLEPERF_H_ */
