/*
 * t3.h - C ABI of the B200 (sm_100a) fused "sliced GEMM + reduce-scatter
 * reduction" library.
 *
 * Problem statement (paper Section 2.4, "Sliced GEMM -> AR", and Section 2.3,
 * ring reduce-scatter): a tensor-parallel sublayer slices its weight along the
 * dot-product dimension over R devices.  Device r computes the partial output
 *     P_r = X_r . W_r          X_r = X[:, r*K_r:(r+1)*K_r],  W_r = W[r*K_r:(r+1)*K_r, :]
 * and a reduce-scatter leaves device c with rows [c*M/R, (c+1)*M/R) of
 *     Y = sum_r P_r .
 * The paper's method (Section 4) starts the reduction of a piece of the output
 * as soon as the producer GEMM has written it, tracked by per-tile counters
 * (Section 4.2.1) whose threshold is "tile size x updates per element", and
 * triggered when the threshold is met (Section 4.2.2).  On one GPU the R
 * devices are simulated as R K-slices: every slice's partial tile is written
 * to a workspace, a counter per output tile counts landed partial tiles, and
 * the R-way sum of a tile (in the ring's order, Section 4.1) runs as soon as
 * its counter reaches its threshold, concurrently with the remaining GEMM
 * tiles.  The sequential baseline (Section 5.3, "Sequential": GEMM kernel,
 * then the collective's kernel) lives in the same library.
 *
 * All pointers named "device" are CUDA device pointers on the device that was
 * current when the plan was made; "host" pointers are ordinary memory.
 * No exceptions cross this boundary.  Functions returning int return 0
 * (T3_OK) or a negative t3_error_t.
 */
#ifndef T3_H_
#define T3_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define T3_VERSION 110

typedef struct t3_plan_s *t3_plan_t;

typedef enum {
    T3_OK = 0,
    T3_ERR_INVALID_ARG = -1,   /* non-positive size, NULL or misaligned pointer, bad enum   */
    T3_ERR_SHAPE = -2,         /* M % R, K % R, (K/R) % 8 or N % 8 is non-zero               */
    T3_ERR_DEVICE = -3,        /* no CUDA device, or its compute capability is not 10.x     */
    T3_ERR_ALLOC = -4,         /* workspace allocation failed                                */
    T3_ERR_CUDA = -5,          /* a CUDA runtime/driver call failed (launch, tensor map ...)  */
    T3_ERR_TIMEOUT = -6,       /* device side: a bounded wait ran out (see t3_plan_status)  */
    T3_ERR_UNSUPPORTED = -7,   /* option combination not available                           */
    T3_ERR_TOO_LARGE = -8      /* size beyond a stated maximum                               */
} t3_error_t;

/* Inputs are always bf16; accumulation and the reduction are fp32. */
typedef enum {
    T3_BF16_OUT_BF16 = 0,      /* Y is bf16 (one round-to-nearest-even at the end) */
    T3_BF16_OUT_F32 = 1        /* Y is fp32 (no final rounding)                    */
} t3_dtype_t;

typedef enum {
    T3_MODE_FUSED = 0,         /* one kernel: GEMM tiles + tracker + concurrent reduction (Sec. 4)   */
    T3_MODE_SEQUENTIAL = 1,    /* GEMM kernel -> full partial buffers -> separate reduce kernel      */
    T3_MODE_GEMM_ONLY = 2,     /* measurement: producer GEMM + partial stores only, Y untouched      */
    T3_MODE_REDUCE_ONLY = 3    /* measurement: the separate reduce kernel over the current partials  */
} t3_mode_t;

/* Storage type of the per-slice partial tiles, i.e. what a device would put on the wire.  fp32 keeps
 * the 1e-4 tolerance of the fp32 output; bf16 follows Section 5.2's 16-bit setup: one extra
 * round-to-nearest-even per slice, the ring sum itself stays fp32, half the reduction traffic. */
typedef enum {
    T3_PARTIAL_F32 = 0,
    T3_PARTIAL_BF16 = 1
} t3_partial_t;

/* Storage of the weight matrix W (mathematically [K,N], Section 2.4).  T3_W_NK: [N][K] row-major,
 * K contiguous, the way a row-parallel Linear keeps its weight (default).  T3_W_KN: [K][N] row-major,
 * N contiguous; needs tile_n to be 128 or 256. */
typedef enum {
    T3_W_NK = 0,
    T3_W_KN = 1
} t3_w_layout_t;

/* Producer schedule.  GROUPED (default): region-major in groups of row tiles, so that a region's R
 * partial tiles are produced close together and its reduction starts early.  STAGGERED: the paper's
 * own order (Section 4.4): in step s the simulated device r produces chunk (r + s + 1) mod R, its
 * own last; kept for study - on one GPU every region completes only during the last step, so the
 * partial tiles live in full buffers and little of the reduction overlaps.  Needs M/R to be a multiple
 * of 256 and clusters of two. */
typedef enum {
    T3_ORDER_GROUPED = 0,
    T3_ORDER_STAGGERED = 1
} t3_order_t;

/* Where the R partial tiles of a region are summed (Section 4.3).
 * T3_REDUCE_RING (default): every slice stores its own fp32 (or bf16) partial tile; once the tracker
 * fires, reducers add the R copies in the chunk's ring order.  Deterministic, 4*R*M*N bytes of
 * partial tiles written and read.
 * T3_REDUCE_INPLACE: the software analog of the paper's near-memory "op-and-store" (Section 4.3; Section
 * 7.4 suggests system-wide atomics on uncached data for hardware without it): every producer tile is
 * ADDED into one fp32 accumulator tile per region by reductions performed at the L2
 * (red.global.add.v4.f32); the tracker then only gates the final pass, which reads the accumulator,
 * rounds once, writes Y and clears the accumulator for the next call.  The workspace shrinks from
 * 4*R*M*N to 4*M*N bytes and the R-way read disappears, but the order in which the R (x split_k)
 * contributions are added is whatever order the tiles finish in: results are NOT bit-reproducible from
 * run to run (they stay within the tolerances; integer-valued inputs stay exact).  Needs fp32 partials
 * and the grouped order.  After a device-side timeout call t3_plan_status before the next call: it
 * clears the half-accumulated tiles. */
typedef enum {
    T3_REDUCE_RING = 0,
    T3_REDUCE_INPLACE = 1
} t3_reduce_t;

/* debug_flags (host-made fault injection for the bounded-wait tests) */
#define T3_DEBUG_INFLATE_EXPECTED 1   /* tracker thresholds +1: the trigger never fires, reducers time out */
#define T3_DEBUG_NO_SPARE_REDUCERS 2  /* SMs without producer tiles stay idle instead of running reducers    */

/*
 * How the output is tiled, tracked and reduced ("address-space configuration",
 * Section 4.4: what to track, at which granularity, trigger condition).
 * Zero in any field selects the default.  NULL selects all defaults.
 * For the fields tile_n, group_tiles, reducer_ctas, reducer_warps, reduce_rows,
 * ring_slots, cluster_ctas, timeout_ms and l2_hints a zero is first replaced
 * by the integer in the environment variable T3_<FIELD NAME IN CAPITALS>
 * (T3_RING_SLOTS, T3_TIMEOUT_MS, ...) when that is set; values a shape does
 * not admit give the usual error code.
 */
typedef struct {
    int32_t mode;            /* t3_mode_t used by t3_gemm_rs                                         */
    int32_t tile_n;          /* output-tile width BN: multiple of 32 in [32,256]; 0 = auto           */
    int32_t group_tiles;     /* schedule group height in 256-row tiles (W reuse vs early trigger)    */
    int32_t reducer_ctas;    /* CTAs (= SMs) that only reduce: the explicit SM split; 0 = none, except */
                             /* that SMs left without producer tiles (fewer tiles than CTA pairs) run  */
                             /* reducers instead of idling                                             */
    int32_t reducer_warps;   /* reducer warps inside each GEMM CTA, 1..8; -1 = none; 0 = auto (8)    */
    int32_t reduce_rows;     /* rows of a reducer work item (a 32-column piece): 32, 16 or 8;        */
                             /* 0 = auto (16 when R > 8, else 32)                                    */
    int32_t stages;          /* shared-memory pipeline depth; 0 = as many as fit                     */
    int32_t timeout_ms;      /* bound on every device-side wait; 0 = 1000                            */
    int32_t debug_flags;     /* T3_DEBUG_*                                                            */
    int32_t max_ctas;        /* cap on the persistent grid; 0 = one CTA per SM                       */
    int32_t ring_slots;      /* fused mode: region slots in the recycled partial ring; 0 = auto (about */
                             /* 64 MB, 40 MB for clusters of four on two-tile groups, never fewer than */
                             /* the regions in flight), -1 = none (full partial buffers), else         */
                             /* >= group_tiles                                                          */
    int32_t cluster_ctas;    /* CTAs per cluster: 2 (one CTA pair) or 4 (two pairs on vertically     */
                             /* adjacent tiles fetch each W k-block once for both; needs a library   */
                             /* built with the shared-fetch TMA file and an even number of 256-row   */
                             /* tiles per schedule group); 0 = auto (4 where possible and            */
                             /* 2*M*N*K >= 1e12 or R >= 16, else 2)                                  */
    int32_t partial_dtype;   /* t3_partial_t: storage type of the partial tiles (the "wire" type)     */
    int32_t w_layout;        /* t3_w_layout_t: how W is stored                                        */
    int32_t order;           /* t3_order_t: the producer schedule                                     */
    int32_t reduce;          /* t3_reduce_t: ring-order sum of stored copies, or update in place      */
    int32_t split_k;         /* producers per (tile, slice): each takes 1/split_k of the slice's      */
                             /* k-blocks and the tracker threshold grows to 2*R*split_k (Section 7.7: */
                             /* split-K producers update an element more than once).  Needs            */
                             /* reduce = T3_REDUCE_INPLACE when > 1; 0 = 1; at most 16 and at most    */
                             /* the slice's k-blocks.  For shapes with too few tiles to fill the GPU  */
                             /* (small M: the token-generation phase, Section 7.3).                  */
    int32_t l2_hints;        /* L2 eviction-priority hints, a bit mask; 0 = auto (3; 39 for clusters of  */
                             /* four on two-tile groups, where a W tile has no reuse once fetched),     */
                             /* -1 = none.  1: X tiles are fetched evict_last; 2: reducers read partial */
                             /* tiles evict_first (their last use); 4 / 8: partial tiles are stored     */
                             /* evict_last / evict_first; 16 / 32: W tiles are fetched evict_last /     */
                             /* evict_first.  Performance only, never results.                          */
    int32_t reserved[2];     /* must be zero                                                         */
} t3_chunking_t;

/* Geometry and cost model of a plan (all host-computed). */
typedef struct {
    int64_t M, N, K;
    int32_t R, K_r;
    int32_t chunk_rows;        /* M / R: rows of one reduce-scatter chunk                    */
    int32_t tile_m, tile_n;    /* output tile = tracker region (Sec. 4.2.1 granularity)      */
    int32_t n_m_tiles, n_n_tiles;
    int32_t n_jobs;            /* producer tiles: n_m_tiles * n_n_tiles * R * split_k        */
    int32_t n_regions;         /* tracked regions = output tiles                             */
    int32_t expected;          /* tracker threshold per region (landed 128-row half tiles)   */
    int32_t group_tiles;
    int32_t ring_slots;        /* 0: fused mode writes the full partial buffers                */
    int32_t grid, gemm_ctas, reducer_ctas, reducer_warps;
    int32_t reduce_rows, n_reduce_items;
    int32_t stages, k_blocks;  /* 64-wide k-blocks per producer tile                         */
    int32_t smem_bytes;
    int32_t mode, dtype;
    int32_t cluster_ctas;      /* 2 or 4, as resolved                                         */
    int32_t partial_dtype;     /* t3_partial_t                                                */
    int32_t w_layout;          /* t3_w_layout_t                                               */
    int32_t order;             /* t3_order_t                                                  */
    int32_t reduce;            /* t3_reduce_t                                                 */
    int32_t split_k;           /* producers per (tile, slice), as resolved                    */
    int32_t tuned;             /* 1 after t3_plan_tune changed or confirmed the configuration */
    int32_t reserved0;
    int64_t workspace_bytes;   /* partial tiles (>= s_p*R*M*N) + ring + counters + control    */
    double flops;              /* 2*M*N*K                                                     */
    double bytes_gemm;         /* 2MK + 2KN + s_p*RMN : operands read once, partials written (s_p = 4 or 2) */
    double bytes_reduce;       /* s_p*RMN + s_y*M*N   : partials read, Y written             */
    double bytes_fused;        /* bytes_gemm + bytes_reduce                                  */
} t3_info_t;

/* Device-side status word, read back by t3_plan_status. */
typedef struct {
    int32_t code;              /* 0 or T3_ERR_TIMEOUT                                        */
    int32_t where;             /* 1 TMA producer, 2 MMA issuer, 3 epilogue, 4 reducer, 5 publisher */
    int32_t block;             /* CTA that gave up first                                     */
    int32_t detail;            /* job or region index it was waiting for                     */
} t3_status_t;

/*
 * t3_plan - configure once, ahead of time (Section 4.4: the tracker and the
 * triggered transfers are "pre-programmed" from the output's address-space
 * configuration).
 *   M, N, K   problem size: X [M,K], W [K,N], Y [M,N]
 *   R         number of simulated tensor-parallel devices = K-slices = chunks
 *   dtype     output type
 *   chunking  host pointer or NULL (defaults); copied
 * Returns a handle owning its device workspace (fp32 partial tiles of all R slices,
 * tracker counters, status word), allocated with cudaMalloc on the current
 * device; NULL on error with the code in t3_last_error().
 * Rejects: sizes <= 0; M % R; K % R; (K/R) % 8; N % 8; device not sm_100.
 */
t3_plan_t t3_plan(int64_t M, int64_t N, int64_t K, int32_t R, t3_dtype_t dtype,
                  const t3_chunking_t *chunking);

/*
 * t3_gemm_rs - the fused op (Sections 4.1-4.2), in the plan's mode.
 *   X  device, bf16 [M,K] row-major                      (read)
 *   W  device, bf16, stored as the plan's w_layout says: [N,K] row-major
 *      (default; K-contiguous per output feature, the mathematical W[k][n]
 *      is W_stored[n][k]) or [K,N] row-major                (read)
 *   Y  device, bf16 or fp32 [M,N] row-major              (written)
 *   stream  a cudaStream_t (NULL = default stream)
 * All three pointers 16-byte aligned, caller-owned, non-overlapping.
 * Asynchronous: work is enqueued on `stream`.  When it completes, rows
 * [c*M/R, (c+1)*M/R) of Y are reduce-scatter chunk c; each element is the sum
 * of the R partial products added in fp32 in the ring order
 * (c-1, c-2, ..., c) mod R (Section 4.1's four-device example).  The result is
 * bit-identical from run to run and between FUSED and SEQUENTIAL modes.
 * One call in flight per plan.  The kernel is persistent (one CTA per SM, all
 * CTA pairs must be resident together because reducers wait on tiles other
 * pairs produce), so two t3 kernels must never share a GPU.  The library
 * sees to that itself: a call made on a different stream than the previous
 * t3 launch on the same device (whatever plan that was) first makes its
 * stream wait, on the GPU and without blocking the host, for the work
 * enqueued so far on that previous stream; calls that follow each other on
 * one stream pay nothing.  Calls from several streams or host threads
 * therefore run one after the other on the GPU.  (Not inside a stream
 * capture: a captured call is ordered by its graph alone.  Not for
 * t3_gemm_rs_static, which creates nothing.  A stream must outlive the next
 * t3 call made on another stream.)
 * The plan must be used with the device it was made on current
 * (T3_ERR_DEVICE otherwise).  Host-detectable errors return a negative code
 * and enqueue nothing; device-side timeouts are reported by t3_plan_status;
 * a timeout left uncollected does not disturb later calls on the plan.
 * In FUSED mode a call enqueues exactly one kernel and nothing else (the
 * kernel re-arms the tracker itself), so calls can be recorded into a CUDA
 * graph by stream capture after one ordinary call per plan and (X, W) pair
 * (the first call with new operand pointers encodes their tensor maps).
 */
int t3_gemm_rs(t3_plan_t plan, const void *X, const void *W, void *Y, void *stream);

/*
 * t3_gemm_rs_ex - t3_gemm_rs with element-wise work fused on the reduced chunk
 * (Section 7.6: the operators that follow the all-reduce - bias, dropout,
 * residual add - can run on the reduce-scattered sub-array, before the
 * all-gather, so each device does 1/R of that work and Y is written once).
 * Per element, in fp32, each step rounded to nearest even and never fused:
 *     y = ((sum_r P_r + bias[n]) * (keep[m][n] ? keep_scale : 0)) + residual[m][n]
 * followed by the single rounding to Y's type.  Steps whose pointer is NULL
 * are skipped; epi == NULL is t3_gemm_rs.  All pointers are device pointers,
 * 16-byte aligned, caller-owned, read only:
 *   bias      [N]    bf16 or fp32 (bias_dtype)
 *   residual  [M,N]  row-major, bf16 or fp32 (residual_dtype); may not alias Y
 *   keep      [M,N]  bytes, non-zero = keep: a dropout mask the CALLER drew
 *                    (the library draws no random numbers); keep_scale is
 *                    the caller's 1/(1-p)
 * Works in every mode that writes Y (the sequential baseline's reduce kernel
 * applies the same tail, so FUSED and SEQUENTIAL stay bit-identical).
 */
typedef enum { T3_EPI_BF16 = 0, T3_EPI_F32 = 1 } t3_epi_dtype_t;
typedef struct {
    const void *bias;
    const void *residual;
    const void *keep;
    float keep_scale;
    int32_t bias_dtype;        /* t3_epi_dtype_t */
    int32_t residual_dtype;    /* t3_epi_dtype_t */
    int32_t reserved;          /* must be zero   */
} t3_epilogue_t;
int t3_gemm_rs_ex(t3_plan_t plan, const void *X, const void *W, void *Y,
                  const t3_epilogue_t *epi /* host or NULL */, void *stream);

/* Same, in an explicit mode (the bench times FUSED, SEQUENTIAL, GEMM_ONLY and
 * REDUCE_ONLY on one plan so that all share one workspace and tile shape;
 * Section 5.3 configurations "Sequential" and the overlap comparison).
 * X, W may be NULL for REDUCE_ONLY; Y may be NULL for GEMM_ONLY. */
int t3_gemm_rs_mode(t3_plan_t plan, int32_t mode, const void *X, const void *W, void *Y,
                    void *stream);

/*
 * t3_gemm_rs_host - the same op for callers whose tensors live in HOST memory
 * (end-to-end path): copies X [M,K] and W (K*N bf16, in the plan's layout) from host to
 * plan-owned device staging buffers, runs t3_gemm_rs in the plan's mode on
 * `stream` and copies Y [M,N] back.
 *   X_host, W_host, Y_host  host pointers, caller-owned; page-locked memory
 *   makes the copies asynchronous, pageable memory makes them synchronous.
 *   X_host and W_host must hold their data when the call is made (the copies
 *   are not ordered after earlier work on `stream`).
 * The copies run on two plan-owned streams, tied to `stream` by events, and
 * alternate between two sets of staging buffers, so that the input copies of
 * one call overlap the kernel and the output copy of the call before it.
 * `stream` waits for the output copy at the end of the call: the result in
 * Y_host is complete once `stream` has been synchronised (or for anything
 * enqueued on `stream` afterwards).  The staging buffers
 * (2 x (2MK + 2KN + s_y*M*N) bytes), streams and events are created on the
 * first call and released by t3_destroy.
 */
int t3_gemm_rs_host(t3_plan_t plan, const void *X_host, const void *W_host, void *Y_host,
                    void *stream);

/*
 * t3_gemm_rs_static - the fused op for callers that must not allocate device memory.
 * (The paper has no counterpart: this is a packaging variant of t3_gemm_rs, not a method step.)
 *
 * Some callers cannot call cudaMalloc: a service thread with a latency bound cannot afford the
 * device-wide synchronisation cudaMalloc / cudaFree imply, a process running under a fixed memory
 * budget has handed all device memory to its own pool, and code in the middle of someone else's
 * stream-ordered pipeline may not disturb that stream's allocator.  t3_plan owns a cudaMalloc'd
 * workspace, so those callers cannot use it.  This call needs no plan: its scratch (the fp32
 * partial tiles of all R slices and the tracker words) lives in one static device array of
 * T3_STATIC_SCRATCH_BYTES that is part of the library image - every GPU that loads the library
 * holds it until the process exits.  The call itself uses no cudaMalloc, cudaFree, or any other
 * allocating routine, on host or device.
 *
 *   M, N, K, R, dtype   as for t3_plan (same shape rules); default tiling, fused mode, partial
 *                       tiles in full buffers (no ring)
 *   X, W, Y             device pointers as for t3_gemm_rs (caller-owned, 16-byte aligned)
 *   stream              a cudaStream_t (NULL = default stream)
 * Errors: the codes of t3_plan / t3_gemm_rs, and T3_ERR_TOO_LARGE when the
 * partial tiles (4*R*M*N bytes, more when M or N are not tile multiples) plus the tracker do not fit T3_STATIC_SCRATCH_BYTES.
 * Result: bit-identical to t3_gemm_rs with default chunking.
 *
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress) and sets
 * the kernel's shared-memory attribute; make that first call outside any stream capture.
 * Every call on a device shares the one array and the array keeps the previous call's contents: the
 * tracker words are cleared on `stream` at the start of each call, the partial tiles are fully
 * rewritten before they are read.  Two calls that overlap on the same GPU (different streams, or
 * different host threads) race on the array and produce garbage; order them yourself.
 * A device-side bounded wait that runs out leaves Y incomplete; this entry point has no status
 * query (use a plan if you need one).
 */
#define T3_STATIC_SCRATCH_BYTES ((32ll << 20) + (64ll << 10))
int t3_gemm_rs_static(int64_t M, int64_t N, int64_t K, int32_t R, t3_dtype_t dtype, const void *X,
                      const void *W, void *Y, void *stream);

/*
 * t3_plan_tune - choose the plan's configuration by measurement (the analog of
 * Section 4.5: the paper's memory-controller arbitration learns its threshold
 * from the producer kernel's behaviour while it runs alone in the first
 * stage; here a short trial on the real operands decides how the reduction
 * shares the GPU with the GEMM).  Runs the op a few times per candidate on
 * `stream`, timing with CUDA events, each timed call after a rewrite of the
 * plan's partial buffers (up to 512 MiB) that sweeps the L2, and keeps the
 * fastest of
 *   { fused with the L2 ring, fused with full partial buffers, sequential }
 *   x reduce_rows { 16, 32 } x cluster_ctas { 2, 4 where available } x group height { g, g/2 }
 * that fit the plan's existing workspace (nothing is allocated).  A candidate
 * replaces the current configuration only if it is at least 3 % faster (5 %
 * if it is the sequential mode).  All
 * candidates produce the same bits, so tuning never changes a result
 * (T3_REDUCE_INPLACE plans: within its stated non-determinism).
 * Synchronous: returns after the trials; Y holds a valid result.  out (host,
 * may be NULL) receives what was tried.  Call it once, before steady-state
 * use and outside stream capture.
 */
typedef struct {
    int32_t n_tried;
    int32_t chosen;              /* index into the arrays below                                   */
    int32_t mode[48], ring_slots[48], reduce_rows[48], cluster_ctas[48], group_tiles[48];
    float us[48];                /* median microseconds per call of each candidate                */
} t3_tune_t;
int t3_plan_tune(t3_plan_t plan, const void *X, const void *W, void *Y, void *stream,
                 t3_tune_t *out /* host or NULL */);

/* t3_destroy - synchronises the device, frees the workspace. NULL is a no-op. */
int t3_destroy(t3_plan_t plan);

/* --- additive queries ----------------------------------------------------- */

/* 1 if this build of the library contains the 4-CTA-cluster kernel variant
 * (cluster_ctas = 4), else 0.  Host only. */
int t3_shared_fetch_available(void);

/* Geometry of a live plan. */
int t3_plan_info(t3_plan_t plan, t3_info_t *out /* host */);

/* Synchronises the plan's last stream, copies the device status word to *out
 * (may be NULL), clears it and re-arms the tracker if a wait had timed out.
 * Returns the status code (0 or T3_ERR_TIMEOUT) or a host error. */
int t3_plan_status(t3_plan_t plan, t3_status_t *out /* host */);

/* Device pointer to, and size of, the full partial buffers (valid until
 * t3_destroy).  The fp32 partial tiles are stored tile by tile in an internal
 * order chosen so that the producer's stores and the reducers' loads cover
 * whole 128-byte lines; the contents are opaque (a test may poison them). */
int t3_plan_partials(t3_plan_t plan, void **partials /* host, receives device ptr */,
                     int64_t *bytes /* host or NULL */);

/* Device pointer to, and size of, the recycled ring of region slots that the
 * FUSED mode writes its partial tiles to (NULL and 0 when the plan has no
 * ring and FUSED uses the full buffers).  Contents opaque; a test may poison
 * it between calls. */
int t3_plan_ring(t3_plan_t plan, void **ring /* host, receives device ptr */,
                 int64_t *bytes /* host or NULL */);

/*
 * t3_plan_timeline - where the time of the plan's last FUSED call went
 * (Section 5.3 compares against an ideal overlap; this splits the fused
 * kernel's own time the same way).  Every CTA records the GPU's global
 * nanosecond timer at four points; the call synchronises the plan's last
 * stream and reduces them:
 *   total_us    first CTA start -> last CTA end
 *   produce_us  first CTA start -> last tracker update (the last partial tile
 *               of the GEMM has landed: the producer phase, run under the
 *               reduction's contention)
 *   tail_us     last tracker update -> last reduced item (reduction that
 *               nothing can overlap with any more)
 *   drain_us    last reduced item -> last CTA end (teardown)
 */
typedef struct {
    double total_us, produce_us, tail_us, drain_us;
    int32_t ctas;
    int32_t reserved;
} t3_timeline_t;
int t3_plan_timeline(t3_plan_t plan, t3_timeline_t *out /* host */);

/* Writes the partial products held in the full partial buffers (as left by
 * the last SEQUENTIAL or GEMM_ONLY call) to dst as plain row-major fp32
 * [R][M][N] (device pointer, caller-owned, 4*R*M*N bytes), asynchronously on
 * `stream`.  Lets a test check the producer GEMM and the reduction stage
 * (Section 2.3's element-wise sum) separately.  T3_ERR_UNSUPPORTED for
 * T3_REDUCE_INPLACE plans (no per-slice copies exist). */
int t3_plan_export_partials(t3_plan_t plan, void *dst /* device */, void *stream);

/* Host-only (no GPU needed): the geometry t3_plan would choose. */
int t3_geometry(int64_t M, int64_t N, int64_t K, int32_t R, t3_dtype_t dtype,
                const t3_chunking_t *chunking, t3_info_t *out /* host */);

/* Host-only: the producer schedule, job j -> (m_tile, n_tile, slice), written
 * as int32 triples to jobs[3*j..]; returns the number of jobs (or a negative
 * code).  Pass jobs = NULL to query the count.  Staggered scheduling analog of
 * Section 4.4: the order decides when each region's trigger can fire. */
int64_t t3_schedule(int64_t M, int64_t N, int64_t K, int32_t R, t3_dtype_t dtype,
                    const t3_chunking_t *chunking, int32_t *jobs /* host */, int64_t max_jobs);

/* Host-only: the reducers' ticket order, item t -> (m_tile, n_tile, row0,
 * n_rows, col0, n_cols) as six int32 each (n_rows = n_cols = 0 for an item
 * that lies wholly in a tile's padding); returns the number of items. */
int64_t t3_reduce_schedule(int64_t M, int64_t N, int64_t K, int32_t R, t3_dtype_t dtype,
                           const t3_chunking_t *chunking, int32_t *items /* host */,
                           int64_t max_items);

/* Host-only: ring summation order of chunk c (Section 4.1 example):
 * order[s] = (c - 1 - s) mod R, ending at c.  `order` has room for R ints. */
int t3_ring_order(int32_t c, int32_t R, int32_t *order /* host */);

/* Host-only: sizeof of the public structs in the order t3_chunking_t, t3_info_t, t3_status_t,
 * t3_epilogue_t, t3_timeline_t, t3_tune_t, written to sizes[0..n) (n <= 6); returns how many exist (6).
 * Lets a foreign-language binding check its struct definitions against the library it loaded. */
int t3_abi_sizes(int32_t *sizes /* host */, int32_t n);

int t3_last_error(void);               /* thread-local code of the last failed call */
const char *t3_strerror(int code);     /* static string                              */
int t3_version(void);

#ifdef __cplusplus
}
#endif
#endif /* T3_H_ */
