// Device code: the fused persistent kernel (TMA producer, tcgen05 MMA issuer,
// epilogue + tracker update, reducers) and the separate reduce kernel of the
// sequential baseline.
//
// The fused kernel runs as CTA pairs.  A pair computes one 256 x BN partial tile
// per job with cta_group::2 MMAs: the CTA with half index h (= cluster rank & 1)
// loads rows [h*128, h*128+128) of the A block and rows [h*BN/2, (h+1)*BN/2) of
// the B block into its own shared memory, the pair's leader (h = 0) issues the
// MMAs for both, and each CTA's 128 accumulator rows land in its own TMEM,
// drained by its own epilogue warps.
//
// The kernel is compiled once per cluster size and per reducer mode (RMode: how a region's stored tiles
// become Y), so that every instantiation holds exactly one variant of the reducers' inner loop.
//
// CLUSTER = 2: one pair per cluster, every CTA fetches its own operands.
// CLUSTER = 4 (built only when the file with the shared-fetch TMA wrapper is
// present): two pairs per cluster work on vertically adjacent tiles (same W
// tile, same slice), so each W k-block is fetched from L2 once for both pairs:
// pair 0's CTAs fetch the even k-blocks and pair 1's the odd ones, each
// delivering its block to the same place in both pairs.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "ptx.cuh"
#include "schedule.h"
#ifdef T3_TMA_SHARED_FETCH
#include "tma_shared_fetch.cuh"
#endif

namespace t3 {

// Four warpgroups: 0 = epilogue (warp w drains TMEM lane quarter w), 1 = service warps (TMA producer,
// MMA issuer, publisher, one idle), 2 and 3 = reducers.  The register file is re-split between them at
// the top of each warpgroup's branch (the kernel is compiled for 128 registers x 512 threads):
// 128 * (REGS_EPILOGUE + REGS_SERVICE) + 256 * REGS_REDUCER <= 65536.
constexpr int REGS_EPILOGUE = 112, REGS_SERVICE = 64, REGS_REDUCER = 168;
constexpr int NUM_THREADS = 512;
constexpr int NUM_WARPS = NUM_THREADS / 32;
// setmaxnreg.inc waits - without a bound - until the CTA's pool holds the registers it asks for, and the
// pool is only what the CTA was launched with (threads x registers per thread at launch, rounded down to
// a multiple of 8) minus what its warps currently hold: a split that adds up to more than that never
// completes.  (Measured the hard way with 640 threads: 96 registers at launch, a split adding up to 64 K.)
constexpr int REGS_AT_LAUNCH = (65536 / NUM_THREADS) / 8 * 8;
static_assert(128 * (REGS_EPILOGUE + REGS_SERVICE) + (NUM_THREADS - 256) * REGS_REDUCER <= NUM_THREADS * REGS_AT_LAUNCH,
              "register re-split exceeds what the CTA is launched with: setmaxnreg.inc would wait forever");
static_assert(NUM_THREADS % 128 == 0, "setmaxnreg is a warpgroup-wide instruction: whole warpgroups only");
constexpr int FIRST_EPI_WARP = 0;
constexpr int TMA_WARP = 4;
constexpr int MMA_WARP = 5;
constexpr int PUB_WARP = 6;
constexpr int FIRST_RED_WARP = 8;
constexpr int MAX_STAGES = 12;
constexpr int TMEM_COLS = 512;          // all of an SM's tensor memory: floor(512 / BN) fp32 accumulators
constexpr int MAX_ACC = 4;             // accumulators in TMEM: floor(512 / BN), 2 for BN = 256, 3 for BN <= 160
constexpr int EPI_CHUNK = 32;                       // accumulator columns drained per epilogue step
constexpr int RED_WARPS_GEMM_CTA = 8;               // reducer warps inside a CTA (warps 8-15)

enum Where { W_TMA = 1, W_MMA = 2, W_EPI = 3, W_RED = 4, W_PUB = 5 };
constexpr int ERR_TIMEOUT = -6;         // = T3_ERR_TIMEOUT

// Element-wise operators applied to the reduced sum before its single rounding (Section 7.6: the work
// that follows the all-reduce - bias, dropout, residual add - done on the reduce-scattered chunk):
//   y = ((sum + bias[n]) * (keep[m][n] ? keep_scale : 0)) + residual[m][n]
// each step one fp32 operation, rounded to nearest even, never contracted.  A NULL pointer skips its step.
struct EpiOps {
    const void* bias;           // [N] bf16 or fp32
    const void* residual;       // [M][N] bf16 or fp32
    const uint8_t* keep;        // [M][N] bytes, non-zero = keep (a dropout mask drawn by the caller)
    float keep_scale;           // 1 / (1 - p)
    int bias_f32, residual_f32;
    int any;                    // 0: nothing to do (plain reduce-scatter)
};

struct alignas(64) KParams {
    CUtensorMap tmX;        // bf16 X viewed as (K_r, R, M)
    CUtensorMap tmW;        // bf16 W[N][K] viewed as (K_r, R, N); or, with w_kn, W[K][N] viewed as (N, K_r, R)
    float* partials;        // [slots][R][tile_elems] fp32 (or bf16, see partial_bf16), tiles in fragment-major order
    int ring_slots;         // 0: one slot per region (full partial buffers, slot = region index);
                            // > 0: the region with sequence number q uses slot q % ring_slots
    long long slot_elems;   // R * tile_elems: a slot holds the R partial tiles of one region
    int tile_elems;         // ROW_BLOCKS * nc * FRAG_ELEMS
    int partial_bf16;       // 1: partial tiles are stored as bf16 (one rounding per slice), summed in fp32 (the host
                            // launches the RMODE_BF16 instantiation; device code looks at its template argument)
    int w_kn;               // 1: W is stored [K][N] (N contiguous): the B operand is MN-major in shared memory
    void* Y;                // [M][N] bf16 or fp32
    uint32_t* counters;     // [n_regions] tracker: landed half tiles per region
    uint32_t* done;         // [n_regions] reduced items per region (frees the region's ring slot)
    uint32_t* ctl;          // [0] reducer ticket, [1] CTAs done, [2] epoch of the launch that is aborting
    int32_t* status;        // [4] code, where, block, detail
    int M, N, R, chunk_rows;
    int BN;
    Sched sched;
    int Kr;                 // K / R: the slice's extent along k
    int k_align;            // 1: k-blocks start on 128-byte lines of X and W rows (see slice_k_shift)
    uint32_t b_bytes;       // per CTA: half B tile bytes of one k-block
    int stages;
    int n_acc, acc_stride;  // accumulators in TMEM and their column pitch
    uint32_t a_bytes, stage_bytes;   // per CTA: A tile bytes of one k-block; a stage = one k-block of A + half B
    int gemm_ctas;          // CTAs [0, gemm_ctas) carry the GEMM roles (even: whole pairs)
    int n_items;            // reducer tickets (0: no reduction in this launch)
    int red_warps;          // reducer warps active in a GEMM CTA
    int out_f32;
    uint32_t expected;      // tracker threshold per region
    unsigned long long timeout_ns;
    uint32_t epoch;         // launch number of the owning plan (> 0): ctl[2] == epoch means "this launch is aborting"
    int split_k;            // producers per (tile, slice): schedule slice index rv = r * split_k + part (in-place mode only when > 1)
    int inplace;            // 1: update-in-place reduction (Section 4.3's analog): the epilogues add every slice's
                            // tile into ONE fp32 accumulator tile per region with L2 reductions; the tracker then
                            // gates only the final convert / store pass, which also clears the accumulator
                            // (the host launches the RMODE_INPLACE instantiation)
    int l2_hints;           // L2 eviction priorities: bit 0: X tiles fetched evict_last; bit 1: reducers read partial
                            // tiles evict_first (their last use); bit 2 / 3: partial tiles stored evict_last /
                            // evict_first; bit 4 / 5: W tiles fetched evict_last / evict_first
    EpiOps epi;             // element-wise work fused on the reduced chunk (Section 7.6)
    unsigned long long* trace;   // [grid][4] globaltimer: start, last tracker update, last reduced item, end; or NULL
};


// k-blocks of slice r.  Slice r starts r * K_r elements into a row; when K_r is not a multiple of 64
// that is not on a 128-byte line for every r, and a 64-wide box would straddle two lines in each row.
// With k_align the blocks of such a slice start `shift` elements before the slice (block b covers
// k in [64 b - shift, 64 b - shift + 64) of the slice), so every box is one whole line per row; the part
// of the first and last box outside the slice is out of the tensor map's bounds and arrives as zeros.
__device__ __forceinline__ int slice_k_shift(const KParams& p, int r) {
    return p.k_align ? (r * p.Kr) & (BK - 1) : 0;
}
__device__ __forceinline__ int slice_k_blocks(const KParams& p, int shift) {
    return (p.Kr + shift + BK - 1) / BK;
}
// A producer job's share of its slice: the schedule's slice index rv names slice r = rv / split_k and
// part rv % split_k of that slice's nkb k-blocks, [kb0, kb1).
__device__ __forceinline__ void job_k_range(const KParams& p, int rv, int& r, int& shift, int& nkb, int& kb0, int& kb1) {
    r = rv;
    shift = slice_k_shift(p, r);
    nkb = slice_k_blocks(p, shift);
    kb0 = 0;
    kb1 = nkb;
    if (p.split_k > 1) {
        r = rv / p.split_k;
        const int part = rv - r * p.split_k;
        shift = slice_k_shift(p, r);
        nkb = slice_k_blocks(p, shift);
        kb0 = part * nkb / p.split_k;
        kb1 = (part + 1) * nkb / p.split_k;
    }
}

// ---------------------------------------------------------------------------
// bounded waits
// ---------------------------------------------------------------------------
// Records the first failure in the status words (kept until the host collects them) and marks THIS launch
// as aborting (ctl[2] = epoch), which is what the other CTAs' waits look at: a status left uncollected by
// an earlier launch does not disturb later ones.
__device__ __forceinline__ void report(const KParams& p, int where, int detail) {
    if (atomicCAS(reinterpret_cast<int*>(p.status), 0, ERR_TIMEOUT) == 0) {
        p.status[1] = where;
        p.status[2] = static_cast<int>(blockIdx.x);
        p.status[3] = detail;
    }
    atomicExch(&p.ctl[2], p.epoch);
    __threadfence();
}
__device__ __forceinline__ bool launch_aborting(const KParams& p) {
    return *reinterpret_cast<volatile uint32_t*>(&p.ctl[2]) == p.epoch;
}

// Returns false when the wait ran out (or the CTA is already aborting).
// CLUSTER: the barrier is arrived on by the peer CTA too (cluster-scope acquire).
template <bool CLUSTER = false>
__device__ __forceinline__ bool mbar_wait(const KParams& p, uint32_t bar, uint32_t parity,
                                          volatile int* abort_flag, int where, int detail) {
    auto try_wait = [&]() { return CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity); };
#pragma unroll 1
    for (int i = 0; i < 128; ++i)
        if (try_wait()) return true;
    const uint64_t t0 = globaltimer_ns();
#pragma unroll 1
    while (true) {
#pragma unroll 1
        for (int i = 0; i < 128; ++i)
            if (try_wait()) return true;
        if (*abort_flag) return false;
        if (globaltimer_ns() - t0 > p.timeout_ns) {
            report(p, where, detail);
            *abort_flag = 1;
            return false;
        }
    }
}

// reducer items of region (mt, nt) that hold at least one element of Y
__device__ __forceinline__ uint32_t region_items(const KParams& p, int mt, int nt) {
    const int prows = min(BMJ, p.M - mt * BMJ), pcols = min(p.BN, p.N - nt * p.BN);
    return static_cast<uint32_t>(((prows + p.sched.reduce_rows - 1) / p.sched.reduce_rows) *
                                 ((pcols + FRAG_COLS - 1) / FRAG_COLS));
}

// Tracker trigger: wait until the region's counter reaches its threshold.
__device__ __forceinline__ bool wait_region(const KParams& p, const uint32_t* cnt, int region) {
#pragma unroll 1
    for (int i = 0; i < 16; ++i)
        if (static_cast<int32_t>(ld_acquire_gpu(cnt) - p.expected) >= 0) return true;
    const uint64_t t0 = globaltimer_ns();
    int polls = 0;
#pragma unroll 1
    while (true) {
        if (static_cast<int32_t>(ld_acquire_gpu(cnt) - p.expected) >= 0) return true;
        __nanosleep(200);
        if ((++polls & 63) == 0) {
            if (launch_aborting(p)) return false;
            if (globaltimer_ns() - t0 > p.timeout_ns) {
                report(p, W_RED, region);
                return false;
            }
        }
    }
}

// ---------------------------------------------------------------------------
// the reduction (Section 2.3's element-wise sum): per element, sequential fp32 adds of the R
// partials in the chunk's ring order.
// ---------------------------------------------------------------------------
// eight neighbouring values of a bf16 or fp32 array, as floats
__device__ __forceinline__ void load_8(const void* base, size_t idx, int is_f32, float (&v)[8]) {
    if (is_f32) {
        const float4* src = reinterpret_cast<const float4*>(static_cast<const float*>(base) + idx);
        const float4 lo = src[0], hi = src[1];
        v[0] = lo.x; v[1] = lo.y; v[2] = lo.z; v[3] = lo.w; v[4] = hi.x; v[5] = hi.y; v[6] = hi.z; v[7] = hi.w;
    } else {
        const uint4 u = *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(base) + idx);
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            v[2 * k] = __uint_as_float(w[k] << 16);
            v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
        }
    }
}

// The element-wise tail of Section 7.6 on one row's eight neighbouring sums (columns col .. col + 7).
__device__ __forceinline__ void apply_epi_8(const EpiOps& eo, int N, int row, int col, float (&v)[8]) {
    const size_t off = static_cast<size_t>(row) * static_cast<size_t>(N) + col;
    // issue the per-element loads first, then the (cached) bias
    uint2 km = make_uint2(0x01010101u, 0x01010101u);
    float res[8];
    if (eo.keep) km = *reinterpret_cast<const uint2*>(eo.keep + off);
    if (eo.residual) load_8(eo.residual, off, eo.residual_f32, res);
    if (eo.bias) {
        float b[8];
        load_8(eo.bias, static_cast<size_t>(col), eo.bias_f32, b);
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = __fadd_rn(v[i], b[i]);
    }
    if (eo.keep) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t byte = ((i < 4 ? km.x : km.y) >> (8 * (i & 3))) & 0xffu;
            v[i] = __fmul_rn(v[i], byte ? eo.keep_scale : 0.0f);
        }
    }
    if (eo.residual) {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = __fadd_rn(v[i], res[i]);
    }
}

// One row's eight neighbouring outputs (columns col .. col + 7): the element-wise tail, if any, then one
// rounding to the output type.
template <bool EPI>
__device__ __forceinline__ void store_y_8(void* Y, int N, int row, int col, const float2 (&a)[4], int out_f32,
                                          const EpiOps& eo) {
    const size_t off = static_cast<size_t>(row) * static_cast<size_t>(N) + col;
    float v[8] = {a[0].x, a[0].y, a[1].x, a[1].y, a[2].x, a[2].y, a[3].x, a[3].y};
    if (EPI && eo.any) apply_epi_8(eo, N, row, col, v);
    if (out_f32) {
        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(Y) + off);
        dst[0] = make_float4(v[0], v[1], v[2], v[3]);
        dst[1] = make_float4(v[4], v[5], v[6], v[7]);
    } else {
        uint4 u;
        __nv_bfloat162 h;
        h = __floats2bfloat162_rn(v[0], v[1]); u.x = *reinterpret_cast<uint32_t*>(&h);
        h = __floats2bfloat162_rn(v[2], v[3]); u.y = *reinterpret_cast<uint32_t*>(&h);
        h = __floats2bfloat162_rn(v[4], v[5]); u.z = *reinterpret_cast<uint32_t*>(&h);
        h = __floats2bfloat162_rn(v[6], v[7]); u.w = *reinterpret_cast<uint32_t*>(&h);
        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(Y) + off) = u;
    }
}

// exchange step of the 4 x 4 transpose among the four lanes of a row (lane bit `S` of q = lane & 3):
// the lane whose bit is clear gives away hi and receives into hi, the other gives lo and receives into lo
template <int S>
__device__ __forceinline__ void quad_exchange(float2& lo, float2& hi, int q) {
    const bool up = (q & S) != 0;
    const float2 send = up ? lo : hi;
    float2 recv;
    recv.x = __shfl_xor_sync(0xffffffffu, send.x, S);
    recv.y = __shfl_xor_sync(0xffffffffu, send.y, S);
    if (up) lo = recv; else hi = recv;
}

// The reduction of 32 x 32 chunks.  Lane 4 g + q works on row g of an 8-row group ("row group" rowsel of
// the chunk): its two float4 (jp = 0, 1) of a stored copy hold columns 8 j + 2 q + {0, 1}, j = 0..3 (slice d's
// copy of the chunk is at chunk + d * slice_stride).  row_base / col_base: global position of the chunk's
// element (0, 0); ncols_left: columns of the chunk that exist (> 0, a multiple of 8).  All 32 lanes must
// call (warp shuffles inside).
// regroups one row's sums among the four lanes of the row and writes its eight neighbouring outputs
template <bool EPI>
__device__ __forceinline__ void finish_row(const float4 (&acc)[2], int q, void* Y, int M, int N, int out_f32, int row, int col_base,
                                           int ncols_left, const EpiOps& eo) {
    float2 a[4] = {make_float2(acc[0].x, acc[0].y), make_float2(acc[0].z, acc[0].w),
                   make_float2(acc[1].x, acc[1].y), make_float2(acc[1].z, acc[1].w)};
    quad_exchange<1>(a[0], a[1], q);
    quad_exchange<1>(a[2], a[3], q);
    quad_exchange<2>(a[0], a[2], q);
    quad_exchange<2>(a[1], a[3], q);
    if (row < M && 8 * q < ncols_left) store_y_8<EPI>(Y, N, row, col_base + 8 * q, a, out_f32, eo);
}

// Sums the R stored copies of row group rowsel in ring order and writes the Y elements that exist; a lane
// keeps 2 x B 128-bit loads in flight.
template <int B, bool EPI>
__device__ __forceinline__ void reduce_row_group(const float* __restrict__ chunk, size_t slice_stride, int rowsel,
                                                 void* Y, int M, int N, int R, int chunk_rows, int out_f32,
                                                 int row_base, int col_base, int ncols_left, int lane, const EpiOps& eo,
                                                 bool last_use, uint64_t pol_first) {
    const int g = lane >> 2, q = lane & 3;
    // float4 index of (rowsel, jp, lane): ((2 * rowsel + jp) * 32 + lane)
    const float* pos = chunk + (static_cast<size_t>(2 * rowsel) * 32 + lane) * 4;
    const int row = row_base + 8 * rowsel + g;
    const int c = min(row, M - 1) / chunk_rows;
    int d = c == 0 ? R - 1 : c - 1;                            // first slice in ring order: (c - 1) mod R
    float4 acc[2];
#pragma unroll 1
    for (int s0 = 0; s0 < R; s0 += B) {
        float4 x[2][B];
#pragma unroll
        for (int i = 0; i < B; ++i)
            if (s0 + i < R) {
                const float* ps = pos + static_cast<size_t>(d) * slice_stride;
                if (last_use) {
                    x[0][i] = ld_partial_v4_hint(ps, pol_first);
                    x[1][i] = ld_partial_v4_hint(ps + 128, pol_first);
                } else {
                    x[0][i] = ld_partial_v4(ps);
                    x[1][i] = ld_partial_v4(ps + 128);
                }
                d = d == 0 ? R - 1 : d - 1;
            }
#pragma unroll
        for (int i = 0; i < B; ++i)
            if (s0 + i < R) {
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    if (s0 + i == 0) {
                        acc[u] = x[u][0];
                    } else {
                        acc[u].x += x[u][i].x; acc[u].y += x[u][i].y; acc[u].z += x[u][i].z; acc[u].w += x[u][i].w;
                    }
                }
            }
    }
    finish_row<EPI>(acc, q, Y, M, N, out_f32, row, col_base, ncols_left, eo);
}

// 16-bit partial tiles: the same reduction of one 8-row group; a lane reads its row's eight values of a
// slice with one 128-bit load (B loads in flight).  chunk points at bf16 storage, slice_stride counts bf16
// elements.
template <int B>
__device__ __forceinline__ void reduce_row_group_bf16(const __nv_bfloat16* __restrict__ chunk, size_t slice_stride,
                                                      int rowsel, void* Y, int M, int N, int R, int chunk_rows,
                                                      int out_f32, int row_base, int col_base, int ncols_left, int lane,
                                                      const EpiOps& eo) {
    const int g = lane >> 2, q = lane & 3;
    const __nv_bfloat16* pos = chunk + (static_cast<size_t>(rowsel) * 32 + lane) * 8;
    const int row = row_base + 8 * rowsel + g;
    const int c = min(row, M - 1) / chunk_rows;
    int d = c == 0 ? R - 1 : c - 1;                            // first slice in ring order: (c - 1) mod R
    float2 a[4];
#pragma unroll 1
    for (int s0 = 0; s0 < R; s0 += B) {
        float4 x[B];
#pragma unroll
        for (int i = 0; i < B; ++i)
            if (s0 + i < R) {
                x[i] = ld_partial_v4(reinterpret_cast<const float*>(pos + static_cast<size_t>(d) * slice_stride));
                d = d == 0 ? R - 1 : d - 1;
            }
#pragma unroll
        for (int i = 0; i < B; ++i)
            if (s0 + i < R) {
                const uint32_t w[4] = {__float_as_uint(x[i].x), __float_as_uint(x[i].y), __float_as_uint(x[i].z), __float_as_uint(x[i].w)};
#pragma unroll
                for (int k = 0; k < 4; ++k) {      // w[k] = the row's columns 8 k + 2 q + {0, 1}
                    const float lo = __uint_as_float(w[k] << 16), hi = __uint_as_float(w[k] & 0xffff0000u);
                    if (s0 + i == 0) {
                        a[k] = make_float2(lo, hi);
                    } else {
                        a[k].x += lo; a[k].y += hi;
                    }
                }
            }
    }
    quad_exchange<1>(a[0], a[1], q);
    quad_exchange<1>(a[2], a[3], q);
    quad_exchange<2>(a[0], a[2], q);
    quad_exchange<2>(a[1], a[3], q);
    if (row < M && 8 * q < ncols_left) store_y_8<true>(Y, N, row, col_base + 8 * q, a, out_f32, eo);
}

// Update-in-place mode: the chunk holds the finished sums.  All row groups [first, end) of the item (at
// most four) are read with their loads in flight together, cleared for the next call, regrouped among
// the four lanes of a row and written to Y.
__device__ __forceinline__ void finish_item_inplace(const float* __restrict__ chunk, int first, int end, void* Y, int M, int N,
                                                    int out_f32, int row_base, int col_base, int ncols_left, int lane,
                                                    const EpiOps& eo) {
    const int g = lane >> 2, q = lane & 3;
    float* pos = const_cast<float*>(chunk) + lane * 4;
    float4 x[4][2];
#pragma unroll
    for (int i = 0; i < 4; ++i)
        if (first + i < end) {
            x[i][0] = ld_partial_v4(pos + static_cast<size_t>(2 * (first + i)) * 128);
            x[i][1] = ld_partial_v4(pos + static_cast<size_t>(2 * (first + i) + 1) * 128);
        }
#pragma unroll
    for (int i = 0; i < 4; ++i)
        if (first + i < end) {
            float* z = pos + static_cast<size_t>(2 * (first + i)) * 128;
            *reinterpret_cast<float4*>(z) = make_float4(0.f, 0.f, 0.f, 0.f);
            *reinterpret_cast<float4*>(z + 128) = make_float4(0.f, 0.f, 0.f, 0.f);
            float2 a[4] = {make_float2(x[i][0].x, x[i][0].y), make_float2(x[i][0].z, x[i][0].w),
                           make_float2(x[i][1].x, x[i][1].y), make_float2(x[i][1].z, x[i][1].w)};
            quad_exchange<1>(a[0], a[1], q);
            quad_exchange<1>(a[2], a[3], q);
            quad_exchange<2>(a[0], a[2], q);
            quad_exchange<2>(a[1], a[3], q);
            const int row = row_base + 8 * (first + i) + g;
            if (row < M && 8 * q < ncols_left) store_y_8<true>(Y, N, row, col_base + 8 * q, a, out_f32, eo);
        }
}

// How a region's stored tiles become Y: a compile-time property of the kernels, so that each instantiation
// holds exactly one variant of the reducers' inner loop and no call.  (Several inlined variants in one
// branch made ptxas spill hundreds of bytes; real calls inside the row-group loop cost the reducers 5-6 %
// on the reduction-heavy shapes because registers then follow the calling convention across the load rounds.)
enum RMode {
    RMODE_RING = 0,        // fp32 partial tiles summed in ring order
    RMODE_RING_EPI = 1,    // the same, then the element-wise tail of Section 7.6
    RMODE_BF16 = 2,        // 16-bit partial tiles (tail at run time)
    RMODE_INPLACE = 3      // update in place: one fp32 accumulator per region (tail at run time)
};

// One reducer item: `rows` (8, 16 or 32) rows of the chunk starting at block row `row_in_block`.
// chunk: the chunk's storage in slice 0 (fp32, or bf16 for RMODE_BF16); slice_stride in elements.
// RMODE_INPLACE: the chunk is the region's single fp32 accumulator (already the sum of all slices): read,
// clear, write Y.
template <int RMODE>
__device__ __forceinline__ void reduce_item(const void* __restrict__ chunk, size_t slice_stride,
                                            int row_in_block, int rows, void* Y, int M, int N, int R, int chunk_rows,
                                            int out_f32, int row_base, int col_base, int ncols_left, int lane,
                                            const EpiOps& eo, int l2_hints) {
    const int first = row_in_block >> 3;
    int end = (row_in_block + rows) >> 3;
    if (row_base + 8 * end > M) end = (M - row_base + 7) >> 3;     // the rest of the block is padding
    if constexpr (RMODE == RMODE_INPLACE) {
        finish_item_inplace(static_cast<const float*>(chunk), first, end, Y, M, N, out_f32, row_base, col_base, ncols_left,
                            lane, eo);
    } else if constexpr (RMODE == RMODE_BF16) {
#pragma unroll 1
        for (int rowsel = first; rowsel < end; ++rowsel)
            reduce_row_group_bf16<8>(static_cast<const __nv_bfloat16*>(chunk), slice_stride, rowsel, Y, M, N, R, chunk_rows,
                                      out_f32, row_base, col_base, ncols_left, lane, eo);
    } else {
        const bool last_use = (l2_hints & 2) != 0;
        const uint64_t pol_first = l2_policy_evict_first();
#pragma unroll 1
        for (int rowsel = first; rowsel < end; ++rowsel)
            reduce_row_group<8, RMODE == RMODE_RING_EPI>(static_cast<const float*>(chunk), slice_stride, rowsel, Y, M, N, R,
                                                         chunk_rows, out_f32, row_base, col_base, ncols_left, lane, eo,
                                                         last_use, pol_first);
    }
}

// Epilogue step: one warp writes its 32 rows x 32 fp32 columns, held in the 16x256b register layout
// (lo: rows 0-15, hi: rows 16-31 of the block), as one 4 KB chunk in fragment-major order: eight
// 128-bit stores per lane, each instruction covering 512 contiguous bytes.
__device__ __forceinline__ void epi_store_frag(const uint32_t (&lo)[16], const uint32_t (&hi)[16], int lane,
                                               float* __restrict__ chunk) {
    float* p0 = chunk + lane * 4;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int rowsel = i >> 1, jp = i & 1, half = rowsel & 1;
        const uint32_t* src = rowsel < 2 ? lo : hi;
        asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p0 + i * 128), "r"(src[8 * jp + 2 * half]),
                     "r"(src[8 * jp + 2 * half + 1]), "r"(src[8 * jp + 4 + 2 * half]), "r"(src[8 * jp + 4 + 2 * half + 1])
                     : "memory");
    }
}
// the same with an L2 eviction-priority policy for the written lines
__device__ __forceinline__ void epi_store_frag_hint(const uint32_t (&lo)[16], const uint32_t (&hi)[16], int lane,
                                                    float* __restrict__ chunk, uint64_t policy) {
    float* p0 = chunk + lane * 4;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int rowsel = i >> 1, jp = i & 1, half = rowsel & 1;
        const uint32_t* src = rowsel < 2 ? lo : hi;
        asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(p0 + i * 128), "r"(src[8 * jp + 2 * half]),
                     "r"(src[8 * jp + 2 * half + 1]), "r"(src[8 * jp + 4 + 2 * half]), "r"(src[8 * jp + 4 + 2 * half + 1]), "l"(policy)
                     : "memory");
    }
}

// Update-in-place variant (Section 4.3's near-memory "op-and-store", done here by the L2's reduction
// units): the same eight 128-bit accesses per lane, each adding its four floats into the region's
// accumulator tile instead of storing them into the slice's own copy.
__device__ __forceinline__ void epi_red_frag(const uint32_t (&lo)[16], const uint32_t (&hi)[16], int lane,
                                             float* __restrict__ chunk) {
    float* p0 = chunk + lane * 4;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int rowsel = i >> 1, jp = i & 1, half = rowsel & 1;
        const uint32_t* src = rowsel < 2 ? lo : hi;
        asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p0 + i * 128),
                     "f"(__uint_as_float(src[8 * jp + 2 * half])), "f"(__uint_as_float(src[8 * jp + 2 * half + 1])),
                     "f"(__uint_as_float(src[8 * jp + 4 + 2 * half])), "f"(__uint_as_float(src[8 * jp + 4 + 2 * half + 1]))
                     : "memory");
    }
}

// The same for 16-bit partial tiles: one round-to-nearest-even per value, four 128-bit stores per lane
// (the eight values a lane holds of one row go out together).
__device__ __forceinline__ void epi_store_frag_bf16(const uint32_t (&lo)[16], const uint32_t (&hi)[16], int lane,
                                                    __nv_bfloat16* __restrict__ chunk) {
    __nv_bfloat16* p0 = chunk + lane * 8;
#pragma unroll
    for (int rowsel = 0; rowsel < 4; ++rowsel) {
        const int half = rowsel & 1;
        const uint32_t* src = rowsel < 2 ? lo : hi;
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {      // k = 2 * jp + (e >> 1): registers 4 k + 2 half + {0, 1}
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(src[4 * k + 2 * half]), __uint_as_float(src[4 * k + 2 * half + 1]));
            w[k] = *reinterpret_cast<const uint32_t*>(&h2);
        }
        asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p0 + rowsel * 256), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3])
                     : "memory");
    }
}

// ---------------------------------------------------------------------------
// fused persistent kernel
// ---------------------------------------------------------------------------
template <int CLUSTER, int RMODE>
__global__ void __cluster_dims__(CLUSTER, 1, 1) __launch_bounds__(NUM_THREADS, 1)
t3_fused_kernel(const __grid_constant__ KParams p) {
    constexpr bool INPLACE = RMODE == RMODE_INPLACE, PARTIAL_BF16 = RMODE == RMODE_BF16;
    static_assert(CLUSTER == 2 || CLUSTER == 4, "one or two CTA pairs per cluster");
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[MAX_STAGES];    // leader's: both CTAs' loads of a stage landed
    __shared__ __align__(8) uint64_t bar_empty[MAX_STAGES];   // own: the MMAs (of every pair of the cluster) reading this stage retired
    __shared__ __align__(8) uint64_t bar_tfull[MAX_ACC];            // own: accumulator complete
    __shared__ __align__(8) uint64_t bar_tempty[MAX_ACC];           // leader's: both CTAs drained the accumulator
    __shared__ __align__(8) uint64_t bar_stored[MAX_ACC];           // own: the four epilogue warps stored their rows of a tile
    __shared__ __align__(8) uint64_t bar_taken[MAX_ACC];            // own: the publisher has seen bar_stored complete
    __shared__ uint32_t tmem_holder;
    __shared__ int abort_flag_s;
    __shared__ int is_last_s;
    __shared__ unsigned long long trace_s[3];                 // kernel start, last tracker update, last reduced item
    volatile int* abort_flag = &abort_flag_s;

    const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x) >> 5, 0);
    const int lane = static_cast<int>(threadIdx.x) & 31;
    const uint32_t rank = cluster_ctarank();
    const uint32_t half = rank & 1u;                          // 0 = leader of its pair
    const uint32_t lead = rank & ~1u;                         // cluster rank of the pair's leader
    const uint32_t pq = rank >> 1;                            // pair within the cluster
    const int pair = static_cast<int>(blockIdx.x) >> 1;
    const int gemm_pairs = p.gemm_ctas >> 1;
    const bool is_gemm = static_cast<int>(blockIdx.x) < p.gemm_ctas;
    const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;

    if (threadIdx.x == 0) {
        abort_flag_s = 0;
        is_last_s = 0;
        trace_s[0] = globaltimer_ns();
        trace_s[1] = 0ull;
        trace_s[2] = 0ull;
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), CLUSTER / CTA_PAIR);
        }
        for (int a = 0; a < MAX_ACC; ++a) {
            mbar_init(smem_u32(&bar_tfull[a]), 1);
            mbar_init(smem_u32(&bar_tempty[a]), EPI_WARPS * CTA_PAIR);
            mbar_init(smem_u32(&bar_stored[a]), EPI_WARPS);
            mbar_init(smem_u32(&bar_taken[a]), 1);
        }
        fence_barrier_init();
        fence_proxy_async_smem();
        if (is_gemm) {
            prefetch_tensormap(&p.tmX);
            prefetch_tensormap(&p.tmW);
        }
    }
    if (warp == MMA_WARP && is_gemm) {
        tmem_alloc_pair(smem_u32(&tmem_holder), TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    cluster_sync_all();                                       // barriers of all CTAs of the cluster are initialised
    tc_fence_after();
    const uint32_t tmem_base = is_gemm ? tmem_holder : 0u;

    if (warp >= 4 && warp < 8) {
      setmaxnreg_dec<REGS_SERVICE>();
      if (is_gemm && warp == TMA_WARP) {
        // ------------------------------------------------ TMA producer (whole warp loops, one lane issues)
        {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            const uint32_t full0 = mapa_cluster(smem_u32(&bar_full[0]), lead);   // the pair leader's full barriers
            const bool hint_x = (p.l2_hints & 1) != 0, hint_w = (p.l2_hints & 48) != 0;
            const uint64_t pol_x = l2_policy_evict_last();
            const uint64_t pol_w = (p.l2_hints & 16) ? l2_policy_evict_last() : l2_policy_evict_first();
            const int a_row_off = static_cast<int>(half) * BM;
            const int b_row_off = static_cast<int>(half) * (p.BN >> 1);
#pragma unroll 1
            for (int j = pair; ok && j < p.sched.n_jobs; j += gemm_pairs) {
                int mt, nt, rv, r, shift, nkb, kb0, kb1;
                decode_job(p.sched, j, mt, nt, rv);
                job_k_range(p, rv, r, shift, nkb, kb0, kb1);
                const int a_row = mt * BMJ + a_row_off, b_row = nt * p.BN + b_row_off;
#pragma unroll 1
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!mbar_wait(p, smem_u32(&bar_empty[s]), ph ^ 1u, abort_flag, W_TMA, j)) {
                        ok = false;
                        break;
                    }
                    // stage layout: [A k-block][half B k-block]
                    const uint32_t dst = tiles + static_cast<uint32_t>(s) * p.stage_bytes;
                    const uint32_t dstB = dst + p.a_bytes;
                    const uint32_t full = full0 + static_cast<uint32_t>(s) * 8u;
                    const int k0 = kb * BK - shift;
                    if (elect_one_sync()) {
                        // a box is counted in full even where it is zero-filled
                        if (half == 0) mbar_arrive_expect_tx(smem_u32(&bar_full[s]), 2u * (p.a_bytes + p.b_bytes));
                        if (hint_x) tma_load_3d_pair_hint(dst, &p.tmX, full, k0, r, a_row, pol_x);
                        else tma_load_3d_pair(dst, &p.tmX, full, k0, r, a_row);
                        // W [N][K]: one box of BN/2 rows x 64 k.  W [K][N]: boxes of 64 k-rows x 64 columns
                        // (128 bytes), 8 KB apart in shared memory.
                        const int nbox = p.w_kn ? (p.BN >> 1) / 64 : 1;
#ifdef T3_TMA_SHARED_FETCH
                        if (CLUSTER == 4) {
                            // the two pairs need the same W block (same rows of W, same slice): they take turns
                            // fetching it for both; the bytes are counted on each destination pair's own barrier
                            if ((kb & 1) == static_cast<int>(pq)) {
                                const uint16_t both = static_cast<uint16_t>(0x5u << half);
                                if (p.w_kn)
                                    for (int bx = 0; bx < nbox; ++bx)
                                        tma_load_3d_pair_shared(dstB + bx * 8192u, &p.tmW, full, b_row + bx * 64, k0, r, both);
                                else if (hint_w)
                                    tma_load_3d_pair_shared_hint(dstB, &p.tmW, full, k0, r, b_row, both, pol_w);
                                else
                                    tma_load_3d_pair_shared(dstB, &p.tmW, full, k0, r, b_row, both);
                            }
                        } else
#endif
                        if (p.w_kn) {
                            for (int bx = 0; bx < nbox; ++bx)
                                tma_load_3d_pair(dstB + bx * 8192u, &p.tmW, full, b_row + bx * 64, k0, r);
                        } else if (hint_w) {
                            tma_load_3d_pair_hint(dstB, &p.tmW, full, k0, r, b_row, pol_w);
                        } else {
                            tma_load_3d_pair(dstB, &p.tmW, full, k0, r, b_row);
                        }
                    }
                    __syncwarp();
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
            }
        }
        __syncwarp();
      } else if (is_gemm && warp == MMA_WARP) {
        // ------------------------------------------------ MMA issuer (the leader CTA's warp loops, one lane issues)
        if (half == 0) {
            const uint32_t idesc = make_idesc_bf16_f32(BMJ, p.BN, p.w_kn != 0);
            const uint16_t pair_mask = static_cast<uint16_t>(0x3u << (2u * pq));       // this pair's two CTAs
            const uint16_t all_mask = static_cast<uint16_t>((1u << CLUSTER) - 1u);     // every CTA that writes into this pair's stages
            const uint64_t a_desc0 = make_sw128_kmajor_desc(tiles);
            // W [K][N]: atoms of 8 k-rows x 64 columns, 1024 bytes apart along K, 8192 bytes (one TMA box) along N;
            // a K = 16 step is two atoms along K
            const uint64_t b_desc0 = p.w_kn ? make_sw128_mnmajor_desc(tiles + p.a_bytes, 8192u, 1024u)
                                            : make_sw128_kmajor_desc(tiles + p.a_bytes);
            const uint64_t b_step = p.w_kn ? 2048u / 16u : 2u;       // descriptor address units per K = 16 step
            const uint32_t stage_units = p.stage_bytes >> 4;          // descriptor address field counts 16 bytes
            int s = 0, jl = 0, acc = 0;
            uint32_t ph = 0, soff = 0, acc_ph = 0;
            bool ok = true;
#pragma unroll 1
            for (int j = pair; ok && j < p.sched.n_jobs; j += gemm_pairs, ++jl) {
                int mt, nt, rv, r, shift, nkb, kb0, kb1;
                decode_job(p.sched, j, mt, nt, rv);
                job_k_range(p, rv, r, shift, nkb, kb0, kb1);
                const int first_step = shift / UMMA_K;                                   // leading all-zero k-steps of block 0
                const int last_steps = (p.Kr + shift - (nkb - 1) * BK + UMMA_K - 1) / UMMA_K;   // k-steps with data in the last block
                if (!mbar_wait<true>(p, smem_u32(&bar_tempty[acc]), acc_ph ^ 1u, abort_flag, W_MMA, j)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * p.acc_stride);
#pragma unroll 1
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!mbar_wait(p, smem_u32(&bar_full[s]), ph, abort_flag, W_MMA, j)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint64_t a_desc = a_desc0 + soff, b_desc = b_desc0 + soff;
                    const int ka = kb == 0 ? first_step : 0;
                    const int kz = kb == nkb - 1 ? last_steps : BK / UMMA_K;
                    if (elect_one_sync()) {
                        // +32 bytes along K inside the 128-byte swizzle row = +2 in the address field
                        if (ka == 0 && kz == BK / UMMA_K) {
                            umma_bf16_ss_pair(d_tmem, a_desc, b_desc, idesc, static_cast<uint32_t>(kb != kb0));
                            umma_bf16_ss_pair(d_tmem, a_desc + 2, b_desc + b_step, idesc, 1u);
                            umma_bf16_ss_pair(d_tmem, a_desc + 4, b_desc + 2 * b_step, idesc, 1u);
                            umma_bf16_ss_pair(d_tmem, a_desc + 6, b_desc + 3 * b_step, idesc, 1u);
                        } else {
                            // first block of a shifted slice (leading zero steps skipped) or the slice's tail block
#pragma unroll 1
                            for (int k = ka; k < kz; ++k)
                                umma_bf16_ss_pair(d_tmem, a_desc + static_cast<uint64_t>(2 * k), b_desc + static_cast<uint64_t>(k) * b_step,
                                                  idesc, static_cast<uint32_t>(kb != kb0 || k != ka));
                        }
                        // the stage is reusable once these MMAs retire: tell every CTA that fetches into it
                        umma_commit_pair_mask(smem_u32(&bar_empty[s]), all_mask);
                        // accumulator complete in both CTAs of the pair
                        if (kb == kb1 - 1) umma_commit_pair_mask(smem_u32(&bar_tfull[acc]), pair_mask);
                    }
                    __syncwarp();
                    soff += stage_units;
                    if (++s == p.stages) { s = 0; ph ^= 1u; soff = 0; }
                }
                if (++acc == p.n_acc) { acc = 0; acc_ph ^= 1u; }
            }
        }
        __syncwarp();
      } else if (is_gemm && warp == PUB_WARP) {
        // ------------------------------------------------ publisher: tracker update (Section 4.2.1)
        // Once the four epilogue warps of this CTA have stored their rows of a partial tile, make the
        // stores visible at gpu scope and bump the region's counter.  The fence has to wait for the
        // stores to drain (microseconds); paying it here keeps it off the epilogue warps.
        {
            int acc = 0;
            uint32_t acc_ph = 0;
#pragma unroll 1
            for (int j = pair; j < p.sched.n_jobs; j += gemm_pairs) {
                int mt, nt, r;
                decode_job(p.sched, j, mt, nt, r);
                if (!mbar_wait(p, smem_u32(&bar_stored[acc]), acc_ph, abort_flag, W_PUB, j)) break;
                if (elect_one_sync()) {
                    mbar_arrive(smem_u32(&bar_taken[acc]));
                    __threadfence();                                   // gpu-scope release of the four warps' stores
                    red_relaxed_gpu_add(&p.counters[mt * p.sched.n_nt + nt], 1u);
                    *reinterpret_cast<volatile unsigned long long*>(&trace_s[1]) = globaltimer_ns();
                }
                __syncwarp();
                if (++acc == p.n_acc) { acc = 0; acc_ph ^= 1u; }
            }
        }
        __syncwarp();
      }
    } else if (warp < FIRST_EPI_WARP + EPI_WARPS) {
      setmaxnreg_dec<REGS_EPILOGUE>();
      if (is_gemm) {
        // ------------------------------------------------ epilogue: TMEM -> partial tile, tracker++
        // Each warp owns 32 accumulator rows and walks them in 32-column chunks; the TMEM load of the
        // next chunk is in flight while the current one is transposed and stored.
        const int q = warp & 3;                                  // TMEM lane quarter this warp may read
        const bool hint_st = (p.l2_hints & 12) != 0 && !PARTIAL_BF16 && !INPLACE;
        const uint64_t pol_st = (p.l2_hints & 4) ? l2_policy_evict_last() : l2_policy_evict_first();
        const uint32_t tempty0 = mapa_cluster(smem_u32(&bar_tempty[0]), lead);   // the pair leader's
        int jl = 0, acc = 0;
        uint32_t acc_ph = 0;
        // slot-availability lookahead for the first tile of this CTA
        const uint32_t* next_slot_done = nullptr;
        uint32_t next_slot_need = 0, next_slot_seen = 0;
        if (p.ring_slots > 0 && pair < p.sched.n_jobs) {
            int m2, n2, r2, seq2;
            decode_job(p.sched, pair, m2, n2, r2, seq2);
            if (seq2 >= p.ring_slots) {
                int pm, pn;
                decode_region(p.sched, seq2 - p.ring_slots, pm, pn);
                next_slot_done = &p.done[pm * p.sched.n_nt + pn];
                next_slot_need = region_items(p, pm, pn);
                next_slot_seen = ld_acquire_gpu(next_slot_done);
            }
        }
#pragma unroll 1
        for (int j = pair; j < p.sched.n_jobs; j += gemm_pairs, ++jl) {
            int mt, nt, r, seq;
            decode_job(p.sched, j, mt, nt, r, seq);
            // ring of region slots: this tile's slot was last used by region seq - ring_slots, which must
            // have been reduced completely.  Its counter was read one tile ago (the read for the next
            // tile is issued now), so the round trip to L2 is off the critical path; normally the value
            // is already final.
            const uint32_t* slot_done = next_slot_done;
            const uint32_t slot_need = next_slot_need, slot_seen = next_slot_seen;
            next_slot_done = nullptr;
            if (p.ring_slots > 0 && j + gemm_pairs < p.sched.n_jobs) {
                int m2, n2, r2, seq2;
                decode_job(p.sched, j + gemm_pairs, m2, n2, r2, seq2);
                if (seq2 >= p.ring_slots) {
                    int pm, pn;
                    decode_region(p.sched, seq2 - p.ring_slots, pm, pn);
                    next_slot_done = &p.done[pm * p.sched.n_nt + pn];
                    next_slot_need = region_items(p, pm, pn);
                    next_slot_seen = ld_acquire_gpu(next_slot_done);
                }
            }
            if (!mbar_wait(p, smem_u32(&bar_tfull[acc]), acc_ph, abort_flag, W_EPI, j)) break;
            tc_fence_after();
            if (slot_done != nullptr && slot_seen < slot_need) {
                const uint64_t t0 = globaltimer_ns();
                bool freed = true;
#pragma unroll 1
                while (ld_acquire_gpu(slot_done) < slot_need) {
                    __nanosleep(100);
                    if (*abort_flag || globaltimer_ns() - t0 > p.timeout_ns) { freed = false; break; }
                }
                if (!freed) {
                    report(p, W_EPI, j);
                    *abort_flag = 1;
                    break;
                }
            }
            __syncwarp();
            const int col0 = nt * p.BN;
            const int ncols = min(p.BN, p.N - col0);
            const int nchunks = (ncols + EPI_CHUNK - 1) / EPI_CHUNK;
            // this warp's row block (half * 4 + q) of slice r's tile in the region's slot
            const int slot = p.ring_slots > 0 ? seq % p.ring_slots : mt * p.sched.n_nt + nt;
            const size_t dst_off = static_cast<size_t>(slot) * static_cast<size_t>(p.slot_elems) +
                                   static_cast<size_t>(INPLACE ? 0 : r) * static_cast<size_t>(p.tile_elems) +
                                   static_cast<size_t>((static_cast<int>(half) * EPI_WARPS + q) * p.sched.nc) * FRAG_ELEMS;
            float* dst = p.partials + dst_off;
            __nv_bfloat16* dst16 = reinterpret_cast<__nv_bfloat16*>(p.partials) + dst_off;
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                   static_cast<uint32_t>(acc * p.acc_stride);
            const uint32_t taddr_hi = taddr + (16u << 16);
            uint32_t alo[16], ahi[16], blo[16], bhi[16];
            tmem_ld_16x256b_x4(taddr, alo);
            tmem_ld_16x256b_x4(taddr_hi, ahi);
#pragma unroll 1
            for (int ci = 0; ci < nchunks; ci += 2) {
                tmem_ld_wait();
                if (ci + 1 < nchunks) {
                    tmem_ld_16x256b_x4(taddr + static_cast<uint32_t>((ci + 1) * EPI_CHUNK), blo);
                    tmem_ld_16x256b_x4(taddr_hi + static_cast<uint32_t>((ci + 1) * EPI_CHUNK), bhi);
                } else {
                    // last TMEM read of this tile is done: hand the accumulator back to the leader's MMA warp
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster_relaxed(tempty0 + static_cast<uint32_t>(acc) * 8u);
                }
                if constexpr (INPLACE) epi_red_frag(alo, ahi, lane, dst + ci * FRAG_ELEMS);
                else if constexpr (PARTIAL_BF16) epi_store_frag_bf16(alo, ahi, lane, dst16 + ci * FRAG_ELEMS);
                else if (hint_st) epi_store_frag_hint(alo, ahi, lane, dst + ci * FRAG_ELEMS, pol_st);
                else epi_store_frag(alo, ahi, lane, dst + ci * FRAG_ELEMS);
                if (ci + 1 < nchunks) {
                    tmem_ld_wait();
                    if (ci + 2 < nchunks) {
                        tmem_ld_16x256b_x4(taddr + static_cast<uint32_t>((ci + 2) * EPI_CHUNK), alo);
                        tmem_ld_16x256b_x4(taddr_hi + static_cast<uint32_t>((ci + 2) * EPI_CHUNK), ahi);
                    } else {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster_relaxed(tempty0 + static_cast<uint32_t>(acc) * 8u);
                    }
                    if constexpr (INPLACE) epi_red_frag(blo, bhi, lane, dst + (ci + 1) * FRAG_ELEMS);
                    else if constexpr (PARTIAL_BF16) epi_store_frag_bf16(blo, bhi, lane, dst16 + (ci + 1) * FRAG_ELEMS);
                    else if (hint_st) epi_store_frag_hint(blo, bhi, lane, dst + (ci + 1) * FRAG_ELEMS, pol_st);
                    else epi_store_frag(blo, bhi, lane, dst + (ci + 1) * FRAG_ELEMS);
                }
            }
            // hand the stored rows to the publisher warp (CTA-scope release: cheap, no drain of the stores)
            if (jl >= p.n_acc && !mbar_wait(p, smem_u32(&bar_taken[acc]), acc_ph ^ 1u, abort_flag, W_EPI, j)) break;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_stored[acc]));
            if (++acc == p.n_acc) { acc = 0; acc_ph ^= 1u; }
        }
        __syncwarp();
      }
    } else {
        setmaxnreg_inc<REGS_REDUCER>();
        // ------------------------------------------------ reducers (triggered by the tracker)
        // A reducer warp draws tickets (items: 16 or 32 rows of one chunk of a region, in completion
        // order), waits for the region's trigger, sums the R stored copies in ring order and writes Y.
        // With a ring of region slots it then reports the item, which frees the slot once all are done.
        const int widx = warp - FIRST_RED_WARP;
        const bool active = p.n_items > 0 && (is_gemm ? widx < p.red_warps : true);
        if (active) {
#pragma unroll 1
            while (true) {
                int t = 0;
                if (lane == 0) t = static_cast<int>(atomicAdd(&p.ctl[0], 1u));
                t = __shfl_sync(0xffffffffu, t, 0);
                if (t >= p.n_items) break;
                const int seq = t / p.sched.items;
                int mt, nt, rb, cc, rib;
                decode_region(p.sched, seq, mt, nt);
                decode_item(p.sched, t - seq * p.sched.items, rb, cc, rib);
                const int row_base = mt * BMJ + rb * FRAG_ROWS;
                const int col_base = nt * p.BN + cc * FRAG_COLS;
                const int ncols_left = min(p.BN, p.N - nt * p.BN) - cc * FRAG_COLS;
                if (row_base + rib >= p.M || ncols_left <= 0) continue;    // nothing of Y in this item
                const int region = mt * p.sched.n_nt + nt;
                if (!wait_region(p, &p.counters[region], region)) break;
                const int slot = p.ring_slots > 0 ? seq % p.ring_slots : region;
                const size_t chunk_off = static_cast<size_t>(slot) * static_cast<size_t>(p.slot_elems) +
                                         static_cast<size_t>(rb * p.sched.nc + cc) * FRAG_ELEMS;
                const void* chunk = PARTIAL_BF16
                                        ? static_cast<const void*>(reinterpret_cast<const __nv_bfloat16*>(p.partials) + chunk_off)
                                        : static_cast<const void*>(p.partials + chunk_off);
                reduce_item<RMODE>(chunk, static_cast<size_t>(p.tile_elems), rib, p.sched.reduce_rows, p.Y, p.M, p.N,
                                   p.R, p.chunk_rows, p.out_f32, row_base, col_base, ncols_left, lane, p.epi, p.l2_hints);
                if (p.ring_slots > 0) {
                    // every lane's loads of this item have returned (their values were used above)
                    __syncwarp();
                    if (lane == 0) red_release_gpu_add(&p.done[region], 1u);
                }
            }
            if (lane == 0) atomicMax(&trace_s[2], static_cast<unsigned long long>(globaltimer_ns()));
        }
        __syncwarp();
    }

    // ------------------------------------------------------ teardown
    if (*abort_flag) {
        // give copies still in flight time to land before shared memory is released
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before();
    cluster_sync_all();            // no CTA of the cluster touches another's barriers, shared memory or TMEM any more
    if (warp == MMA_WARP && is_gemm) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
    // the last CTA to finish re-arms the tracker for the next call
    if (threadIdx.x == 0) {
        if (p.trace != nullptr) {
            unsigned long long* t = p.trace + 4ull * blockIdx.x;
            t[0] = trace_s[0]; t[1] = trace_s[1]; t[2] = trace_s[2]; t[3] = globaltimer_ns();
        }
        __threadfence();
        const uint32_t done = atomicAdd(&p.ctl[1], 1u);
        if (done == gridDim.x - 1) {
            __threadfence();
            is_last_s = 1;
        }
    }
    __syncthreads();
    if (is_last_s) {
        for (int i = threadIdx.x; i < p.sched.n_regions; i += NUM_THREADS) {
            p.counters[i] = 0u;
            p.done[i] = 0u;
        }
        if (threadIdx.x == 0) {
            p.ctl[0] = 0u;
            p.ctl[1] = 0u;
        }
    }
}

// ---------------------------------------------------------------------------
// sequential baseline: the separate reduce kernel over full partial buffers (slot = region index)
// ---------------------------------------------------------------------------
template <int RMODE>       // compiled once per reducer mode, so that each keeps two blocks per SM
__global__ void __launch_bounds__(256, 2) t3_reduce_kernel(const float* __restrict__ partials, void* Y, int M, int N, int R,
                                                           int chunk_rows, int out_f32, int BN, Sched sched,
                                                           long long slot_elems, int tile_elems, EpiOps epi) {
    constexpr bool partial_bf16 = RMODE == RMODE_BF16;
    const int lane = static_cast<int>(threadIdx.x) & 31;
    const long long warps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    const long long n_items = static_cast<long long>(sched.n_regions) * sched.items;
#pragma unroll 1
    for (long long t = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); t < n_items; t += warps) {
        const int region = static_cast<int>(t / sched.items);
        const int mt = region / sched.n_nt, nt = region - mt * sched.n_nt;
        int rb, cc, rib;
        decode_item(sched, static_cast<int>(t - static_cast<long long>(region) * sched.items), rb, cc, rib);
        const int row_base = mt * BMJ + rb * FRAG_ROWS;
        const int col_base = nt * BN + cc * FRAG_COLS;
        const int ncols_left = min(BN, N - nt * BN) - cc * FRAG_COLS;
        if (row_base + rib >= M || ncols_left <= 0) continue;
        const size_t chunk_off = static_cast<size_t>(region) * static_cast<size_t>(slot_elems) +
                                 static_cast<size_t>(rb * sched.nc + cc) * FRAG_ELEMS;
        const void* chunk = partial_bf16 ? static_cast<const void*>(reinterpret_cast<const __nv_bfloat16*>(partials) + chunk_off)
                                         : static_cast<const void*>(partials + chunk_off);
        reduce_item<RMODE>(chunk, static_cast<size_t>(tile_elems), rib, sched.reduce_rows, Y, M, N, R, chunk_rows,
                           out_f32, row_base, col_base, ncols_left, lane, epi, 0);
    }
}

// verification aid: the full partial buffers rewritten as plain row-major [R][M][N]
__global__ void __launch_bounds__(256) t3_export_partials_kernel(const float* __restrict__ partials, float* __restrict__ dst,
                                                                 int M, int N, int R, int BN, Sched sched,
                                                                 long long slot_elems, int tile_elems, int partial_bf16) {
    const long long total = static_cast<long long>(R) * M * N;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int n = static_cast<int>(i % N);
        const long long rm = i / N;
        const int m = static_cast<int>(rm % M), r = static_cast<int>(rm / M);
        const int mt = m / BMJ, nt = n / BN;
        const long long off = static_cast<long long>(mt * sched.n_nt + nt) * slot_elems + static_cast<long long>(r) * tile_elems +
                              frag_offset(m - mt * BMJ, n - nt * BN, sched.nc, partial_bf16 != 0);
        dst[i] = partial_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(partials)[off]) : partials[off];
    }
}

}  // namespace t3
