// Host side of the C ABI declared in include/t3.h: argument validation, plan
// geometry (tile shape, schedule, tracker thresholds, SM split), tensor maps,
// workspace ownership and kernel launches.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>

#include "../../include/t3.h"
#include "kernels.cuh"

namespace {

thread_local int g_last_error = 0;
constexpr uint32_t PLAN_MAGIC = 0x54335031u;  // "T3P1"
constexpr int DEFAULT_SMS = 148;              // B200; used only by the host-only queries
constexpr int SMEM_LIMIT = 232448;            // 227 KB opt-in maximum per CTA on sm_100
constexpr int SMEM_STATIC_SLACK = 512;        // barriers and flags declared statically in the kernel
#ifdef T3_TMA_SHARED_FETCH
constexpr bool HAVE_SHARED_FETCH = true;
#else
constexpr bool HAVE_SHARED_FETCH = false;
#endif

int fail(int code) {
    g_last_error = code;
    return code;
}

// One rank of a multi-process launch (torchrun and the like export WORLD_SIZE / LOCAL_WORLD_SIZE): the
// kernel variant whose W fetches are multicast TMA loads is for one process on one GPU only.
bool multi_process_launch() {
    for (const char* key : {"WORLD_SIZE", "LOCAL_WORLD_SIZE"}) {
        const char* v = std::getenv(key);
        if (v && *v && std::atoi(v) != 1) return true;
    }
    return false;
}

struct Geometry {
    int ring_slots;           // 0 = full partial buffers in every mode
    int64_t slot_elems;       // R * tile_elems: the R partial tiles of one region
    int tile_elems;           // floats of one stored partial tile (fragment-major, padded to 32-column chunks)
    int64_t partial_bytes;    // full partial buffers: one slot per region
    t3_chunking_t cfg;   // resolved
    t3_info_t info;
    t3::Sched sched;
    int k_align;              // k-blocks may start on 128-byte lines (row pitch is a multiple of 128 bytes)
    uint32_t a_bytes, b_bytes, stage_bytes;
    int spare_reducers;       // reducer-only CTAs added on SMs that have no producer tiles (part of info.reducer_ctas)
};

// A field the caller left at 0 (= automatic) takes its value from the environment variable `name` when that
// is set to an integer: a way to steer the automatic choices of code that passes NULL for the chunking.
void env_default(int32_t& field, const char* name) {
    if (field != 0) return;
    const char* v = std::getenv(name);
    if (!v || !*v) return;
    char* end = nullptr;
    const long x = std::strtol(v, &end, 10);
    if (end != v && *end == 0 && x >= -1 && x <= 1 << 20) field = static_cast<int32_t>(x);
}

int pick_tile_n(int64_t N, int step) {
    // multiple of `step` in [128,256] with the least padded width; ties -> widest
    int best = 256;
    int64_t best_pad = -1;
    for (int bn = 256; bn >= 128; bn -= step) {
        const int64_t padded = (N + bn - 1) / bn * bn;
        if (best_pad < 0 || padded < best_pad) {
            best_pad = padded;
            best = bn;
        }
    }
    if (N < 128) best = static_cast<int>((N + step - 1) / step * step);
    return best;
}

int floor_pow2(int v) {
    int p = 1;
    while (2 * p <= v) p *= 2;
    return p;
}

int resolve_geometry(int64_t M, int64_t N, int64_t K, int32_t R, int dtype, const t3_chunking_t* in,
                     int sm_count, Geometry& g) {
    if (M <= 0 || N <= 0 || K <= 0 || R <= 0) return T3_ERR_INVALID_ARG;
    if (dtype != T3_BF16_OUT_BF16 && dtype != T3_BF16_OUT_F32) return T3_ERR_INVALID_ARG;
    if (M % R || K % R) return T3_ERR_SHAPE;
    const int64_t Kr = K / R;
    if (Kr % 8 || N % 8) return T3_ERR_SHAPE;
    if (M > (1ll << 30) || N > (1ll << 30) || K > (1ll << 30) || R > 128) return T3_ERR_TOO_LARGE;
    if (M * N / 4 >= (1ll << 31)) return T3_ERR_TOO_LARGE;

    t3_chunking_t c;
    std::memset(&c, 0, sizeof c);
    if (in) c = *in;
    if (c.reserved[0] != 0 || c.reserved[1] != 0) return T3_ERR_INVALID_ARG;
    env_default(c.tile_n, "T3_TILE_N");
    env_default(c.group_tiles, "T3_GROUP_TILES");
    env_default(c.reducer_ctas, "T3_REDUCER_CTAS");
    env_default(c.reducer_warps, "T3_REDUCER_WARPS");
    env_default(c.reduce_rows, "T3_REDUCE_ROWS");
    env_default(c.ring_slots, "T3_RING_SLOTS");
    env_default(c.cluster_ctas, "T3_CLUSTER_CTAS");
    env_default(c.timeout_ms, "T3_TIMEOUT_MS");
    env_default(c.l2_hints, "T3_L2_HINTS");
    if (c.l2_hints < -1 || c.l2_hints > 63 || (c.l2_hints > 0 && ((c.l2_hints & 12) == 12 || (c.l2_hints & 48) == 48))) return T3_ERR_INVALID_ARG;
    const bool l2_auto = c.l2_hints == 0;      // resolved once the cluster size is known
    if (c.reduce != T3_REDUCE_RING && c.reduce != T3_REDUCE_INPLACE) return T3_ERR_INVALID_ARG;
    if (c.order != T3_ORDER_GROUPED && c.order != T3_ORDER_STAGGERED) return T3_ERR_INVALID_ARG;
    if (c.w_layout != T3_W_NK && c.w_layout != T3_W_KN) return T3_ERR_INVALID_ARG;
    if (c.partial_dtype != T3_PARTIAL_F32 && c.partial_dtype != T3_PARTIAL_BF16) return T3_ERR_INVALID_ARG;
    if (c.cluster_ctas != 0 && c.cluster_ctas != 2 && c.cluster_ctas != 4) return T3_ERR_INVALID_ARG;
    if (c.mode < T3_MODE_FUSED || c.mode > T3_MODE_REDUCE_ONLY) return T3_ERR_INVALID_ARG;
    if (c.split_k == 0) c.split_k = 1;
    if (c.split_k < 1 || c.split_k > 16) return T3_ERR_INVALID_ARG;
    if (c.split_k > 1 && c.reduce != T3_REDUCE_INPLACE) return T3_ERR_UNSUPPORTED;
    if (c.reduce == T3_REDUCE_INPLACE && (c.partial_dtype != T3_PARTIAL_F32 || c.order != T3_ORDER_GROUPED)) return T3_ERR_UNSUPPORTED;

    if (c.tile_n == 0) c.tile_n = pick_tile_n(N, c.w_layout == T3_W_KN ? 128 : 32);
    if (c.tile_n < 32 || c.tile_n > 256 || c.tile_n % 32) return T3_ERR_INVALID_ARG;
    // W stored [K][N] is fetched in boxes of 64 columns per CTA: each CTA's half tile must be whole boxes
    if (c.w_layout == T3_W_KN && c.tile_n % 128) return T3_ERR_INVALID_ARG;

    const int64_t n_mt64 = (M + t3::BMJ - 1) / t3::BMJ;
    const int64_t n_nt64 = (N + c.tile_n - 1) / c.tile_n;
    if (c.split_k > (Kr + t3::BK - 1) / t3::BK) return T3_ERR_INVALID_ARG;     // every producer needs a k-block
    const int Rv = R * c.split_k;                   // producers per output tile ("virtual slices")
    const bool inplace = c.reduce == T3_REDUCE_INPLACE;
    const int copies = inplace ? 1 : R;             // stored tiles per region: one accumulator, or one copy per slice
    if (n_mt64 * n_nt64 * Rv > (1ll << 30)) return T3_ERR_TOO_LARGE;
    const int n_mt = static_cast<int>(n_mt64), n_nt = static_cast<int>(n_nt64);

    if (c.group_tiles < 0) return T3_ERR_INVALID_ARG;
    if (c.group_tiles == 0) {
        // keep one group's X rows (G*256 x K bf16) well inside L2 while W tiles are reused G times
        int64_t gmax = (48ll << 20) / (512 * K);
        if (gmax < 1) gmax = 1;
        if (gmax > 8) gmax = 8;
        c.group_tiles = floor_pow2(static_cast<int>(gmax));
        // ... and keep the ring of region slots that this group height needs (regions in production plus
        // two groups, see the ring sizing below) within about half of L2: with many slices a slot is large
        // (R = 16, BN = 256: 4 MB) and a group of 8 would ask for a 100 MB ring (measured: 247 -> 203 us on
        // R = 16, M = 4096, H = 2048 with groups of 4)
        const int64_t slot_b = static_cast<int64_t>(copies) * t3::ROW_BLOCKS * ((c.tile_n + t3::FRAG_COLS - 1) / t3::FRAG_COLS) *
                               t3::FRAG_ELEMS * (c.partial_dtype == T3_PARTIAL_BF16 ? 2 : 4);
        while (c.group_tiles > 1 && ((sm_count + Rv - 1) / Rv + 2ll * c.group_tiles) * slot_b > (72ll << 20)) c.group_tiles /= 2;
    }
    if (c.group_tiles > n_mt) c.group_tiles = n_mt;

    if (c.max_ctas < 0) return T3_ERR_INVALID_ARG;
    {
        // Two pairs per cluster work on jobs j, j + 1 (j even): these must be vertically adjacent tiles of
        // one W tile and one slice, which holds when every schedule group has an even number of row tiles.
        const bool can4 = HAVE_SHARED_FETCH && !multi_process_launch() && c.order == T3_ORDER_GROUPED && n_mt % 2 == 0 && c.group_tiles % 2 == 0 && sm_count >= 4 &&
                          (c.max_ctas == 0 || c.max_ctas >= 4) && c.reducer_ctas % 4 == 0;
        if (c.cluster_ctas == 4 && !can4) return T3_ERR_UNSUPPORTED;
        // Clusters of four fit on fewer SMs (132 of 148 on a B200) but fetch W from L2 once per two pairs;
        // measured over the shape sweep, that pays for long, power-limited problems and for R >= 16.
        const double flops = 2.0 * static_cast<double>(M) * static_cast<double>(N) * static_cast<double>(K);
        if (c.cluster_ctas == 0) c.cluster_ctas = (can4 && (flops >= 1e12 || R >= 16)) ? 4 : 2;
    }
    const int cl = c.cluster_ctas;
    // L2 eviction priorities, measured (interleaved timings and DRAM-traffic captures): X tiles kept (a schedule
    // group's X rows are reused by every column tile) and partial tiles released by the reducers' reads are
    // worth 2-6 % everywhere.  In clusters of four both row tiles that use a W tile sit in the same cluster, so
    // W lines have no further use once fetched: marking them evict_first, and the partial tiles evict_last
    // until they are read, lets the ring of region slots survive in L2 (large FC-2 shape scaled to 1 024 rows:
    // 2.37 -> 1.37 GB of DRAM traffic per launch).  That holds for two-tile groups only; taller groups (and
    // pairs) reuse a W tile across the group's row tiles, and there W evict_first costs 5-20 %.
    if (l2_auto) c.l2_hints = (cl == 4 && c.group_tiles == 2) ? 39 : 3;
    int grid = sm_count / cl * cl;                 // whole clusters
    if (c.max_ctas > 0 && c.max_ctas < grid) grid = c.max_ctas / cl * cl;
    if (grid < cl) return T3_ERR_INVALID_ARG;
    if (c.reducer_ctas < 0 || (c.reducer_ctas % cl) || c.reducer_ctas >= grid) return T3_ERR_INVALID_ARG;
    if (c.reducer_warps == 0) c.reducer_warps = t3::RED_WARPS_GEMM_CTA;
    if (c.reducer_warps == -1) c.reducer_warps = 0;
    if (c.reducer_warps < 0 || c.reducer_warps > t3::RED_WARPS_GEMM_CTA) return T3_ERR_INVALID_ARG;
    if (c.reducer_warps == 0 && c.reducer_ctas == 0 && c.mode == T3_MODE_FUSED) return T3_ERR_INVALID_ARG;
    // Measured: whole chunks amortise the per-item cost (ticket, trigger poll, release); with more than 8
    // slices an 8-row group takes two rounds of loads, and half-chunk items keep the tail and the slot
    // turn-around short.
    if (c.reduce_rows == 0) c.reduce_rows = R > 8 ? t3::FRAG_ROWS / 2 : t3::FRAG_ROWS;
    if (c.reduce_rows != 32 && c.reduce_rows != 16 && c.reduce_rows != 8) return T3_ERR_INVALID_ARG;
    if (c.timeout_ms == 0) c.timeout_ms = 1000;
    if (c.timeout_ms < 0 || c.timeout_ms > 60000) return T3_ERR_INVALID_ARG;

    const uint32_t a_bytes = t3::BM * t3::BK * 2;
    const uint32_t b_bytes = static_cast<uint32_t>(c.tile_n / t3::CTA_PAIR) * t3::BK * 2;   // per CTA, per k-block
    const uint32_t stage_bytes = a_bytes + b_bytes;                                         // one k-block of A and of half B
    const int epi_bytes = 0;   // the epilogue stores straight from registers
    const int red_bytes = 0;   // reducers work from registers
    const int max_stages =
        (SMEM_LIMIT - SMEM_STATIC_SLACK - 1024 - epi_bytes - red_bytes) / static_cast<int>(stage_bytes);
    if (c.stages == 0) c.stages = max_stages < t3::MAX_STAGES ? max_stages : t3::MAX_STAGES;
    if (c.stages < 2 || c.stages > t3::MAX_STAGES || c.stages > max_stages) return T3_ERR_INVALID_ARG;

    g.cfg = c;
    g.spare_reducers = 0;
    g.a_bytes = a_bytes;
    g.b_bytes = b_bytes;
    g.stage_bytes = stage_bytes;
    g.sched = t3::make_sched(n_mt, n_nt, Rv, c.group_tiles, c.reduce_rows, c.tile_n);
    if (c.order == T3_ORDER_STAGGERED) {
        // device r's chunk of a step must be whole row tiles
        if ((M / R) % t3::BMJ) return T3_ERR_UNSUPPORTED;
        g.sched.staggered = 1;
        g.sched.tpc = static_cast<int>((M / R) / t3::BMJ);
        c.ring_slots = -1;             // every region stays open until the last step: nothing to recycle
        g.cfg.ring_slots = -1;
    }
    // Slices whose first element is not on a 128-byte line of its row get their k-blocks shifted onto line
    // boundaries (possible when every row starts on a line: K a multiple of 64; the operand pointers are
    // checked per call).  The shifted slices may need one k-block more.
    g.k_align = (K % t3::BK == 0 && Kr % t3::BK != 0) ? 1 : 0;
    int max_shift = 0;
    if (g.k_align)
        for (int r = 0; r < R; ++r) {
            const int sh = static_cast<int>((static_cast<int64_t>(r) * Kr) % t3::BK);
            if (sh > max_shift) max_shift = sh;
        }
    const int nkb = static_cast<int>((Kr + max_shift + t3::BK - 1) / t3::BK);

    t3_info_t& o = g.info;
    std::memset(&o, 0, sizeof o);
    o.M = M; o.N = N; o.K = K; o.R = R; o.K_r = static_cast<int32_t>(Kr);
    o.chunk_rows = static_cast<int32_t>(M / R);
    o.tile_m = t3::BMJ; o.tile_n = c.tile_n;
    o.n_m_tiles = n_mt; o.n_n_tiles = n_nt;
    o.n_jobs = g.sched.n_jobs;
    o.n_regions = g.sched.n_regions;
    // Section 4.2.1: threshold = (tile size) x (updates per element); the unit counted here is one
    // CTA's 128-row half of the tile, and every one of the R slices updates each element once (split_k
    // times when a slice's product is itself split along k, Section 7.7).
    o.expected = t3::CTA_PAIR * Rv + ((c.debug_flags & T3_DEBUG_INFLATE_EXPECTED) ? 1 : 0);
    o.group_tiles = c.group_tiles;
    o.grid = grid;
    o.reducer_ctas = c.reducer_ctas;
    o.gemm_ctas = grid - c.reducer_ctas;
    if (o.gemm_ctas > t3::CTA_PAIR * o.n_jobs) {
        // fewer producer tiles than CTA pairs (small M: Section 7.3's generation phase, or a tiny problem):
        // the SMs left over run reducers only instead of idling, which shortens the reduction that starts
        // when the one wave of tiles lands
        o.gemm_ctas = t3::CTA_PAIR * o.n_jobs;
        if (c.mode == T3_MODE_FUSED && c.reducer_ctas == 0 && !(c.debug_flags & T3_DEBUG_NO_SPARE_REDUCERS)) {
            g.spare_reducers = (grid - o.gemm_ctas) / cl * cl;
            o.reducer_ctas = g.spare_reducers;
        }
    }
    o.grid = o.gemm_ctas + o.reducer_ctas;
    o.reducer_warps = c.reducer_warps;
    o.reduce_rows = c.reduce_rows;
    if (static_cast<int64_t>(g.sched.n_regions) * g.sched.items > (1ll << 30)) return T3_ERR_TOO_LARGE;
    o.n_reduce_items = g.sched.n_regions * g.sched.items;
    o.stages = c.stages;
    o.k_blocks = nkb;
    o.smem_bytes = c.stages * static_cast<int>(stage_bytes) + epi_bytes + red_bytes + 1024;
    g.tile_elems = t3::ROW_BLOCKS * g.sched.nc * t3::FRAG_ELEMS;
    g.slot_elems = static_cast<int64_t>(copies) * g.tile_elems;
    const int esize = c.partial_dtype == T3_PARTIAL_BF16 ? 2 : 4;
    g.partial_bytes = static_cast<int64_t>(g.sched.n_regions) * g.slot_elems * esize;
    {
        // Ring of region slots for the fused mode: a slot holds the R partial tiles of one region and is
        // reused once that region has been reduced, so the partial traffic stays in L2.
        // Deadlock freedom needs ring_slots >= group_tiles (all tiles of the region that used the slot
        // before then precede this tile in the schedule); more slots only avoid stalls.
        const int64_t slot_bytes = g.slot_elems * esize;
        const int pairs = (grid - c.reducer_ctas) / t3::CTA_PAIR;
        int64_t want = c.ring_slots;
        if (want == 0) {
            // about half of the 126 MB L2; a third where W streams through with no reuse (clusters of four on
            // two-tile groups): the ring then stays resident beside the group's X rows (measured on the large
            // FC-2 shape: 16 slots of 4 MB spill to DRAM entirely, 8-10 stay, 6 stall the producers)
            const int64_t target = (cl == 4 && c.group_tiles == 2) ? (40ll << 20) : (64ll << 20);
            want = target / slot_bytes;
            // regions in production (one per R jobs in flight) plus two groups' worth waiting for reducers
            const int64_t in_flight = (pairs + Rv - 1) / Rv + 2ll * c.group_tiles + 1;
            if (want < in_flight) want = in_flight;
        }
        if (want < 0) want = 0;                                   // -1: full partial buffers in fused mode too
        if (want > 0 && want < c.group_tiles) return T3_ERR_INVALID_ARG;
        if (want >= g.sched.n_regions) want = 0;                  // everything fits: no recycling needed
        g.ring_slots = static_cast<int>(want);
        o.ring_slots = g.ring_slots;
    }
    o.mode = c.mode;
    o.dtype = dtype;
    o.cluster_ctas = cl;
    o.partial_dtype = c.partial_dtype;
    o.w_layout = c.w_layout;
    o.order = c.order;
    o.reduce = c.reduce;
    o.split_k = c.split_k;
    const double sy = dtype == T3_BF16_OUT_F32 ? 4.0 : 2.0;
    const double dM = static_cast<double>(M), dN = static_cast<double>(N), dK = static_cast<double>(K);
    o.workspace_bytes = g.partial_bytes + static_cast<int64_t>(4) * (2 * o.n_regions + 64) +
                        static_cast<int64_t>(g.ring_slots) * g.slot_elems * esize;
    o.flops = 2.0 * dM * dN * dK;
    // update in place: every producer tile still ships 4 bytes per element (to the L2's reduction units); the
    // final pass reads the accumulator once, clears it and writes Y
    o.bytes_gemm = 2.0 * dM * dK + 2.0 * dK * dN + static_cast<double>(esize) * Rv * dM * dN;
    o.bytes_reduce = inplace ? (8.0 + sy) * dM * dN : static_cast<double>(esize) * R * dM * dN + sy * dM * dN;
    o.bytes_fused = o.bytes_gemm + o.bytes_reduce;
    return T3_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 matrix [rows][K] (K contiguous) viewed per K-slice: (k in slice, slice, row).
// A k-block that overruns the slice reads zeros, not the next slice.
int encode_sliced_map(CUtensorMap* out, const void* base, int64_t rows, int64_t K, int R, int box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return T3_ERR_CUDA;
    const int64_t Kr = K / R;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(Kr), static_cast<cuuint64_t>(R), static_cast<cuuint64_t>(rows)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(Kr) * 2, static_cast<cuuint64_t>(K) * 2};
    cuuint32_t box[3] = {static_cast<cuuint32_t>(t3::BK), 1u, static_cast<cuuint32_t>(box_rows)};
    cuuint32_t estr[3] = {1u, 1u, 1u};
    CUresult rc = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS ? T3_OK : T3_ERR_CUDA;
}

// bf16 matrix [K][N] (N contiguous) viewed per K-slice: (column, k in slice, slice); boxes of 64 columns
// (one 128-byte swizzle row) x 64 k-rows.  Rows outside the slice read zeros.
int encode_kn_map(CUtensorMap* out, const void* base, int64_t N, int64_t K, int R) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return T3_ERR_CUDA;
    const int64_t Kr = K / R;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(Kr), static_cast<cuuint64_t>(R)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(N) * 2, static_cast<cuuint64_t>(Kr) * static_cast<cuuint64_t>(N) * 2};
    cuuint32_t box[3] = {64u, static_cast<cuuint32_t>(t3::BK), 1u};
    cuuint32_t estr[3] = {1u, 1u, 1u};
    CUresult rc = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS ? T3_OK : T3_ERR_CUDA;
}

int encode_w_map(CUtensorMap* out, const void* W, const t3_info_t& o) {
    if (o.w_layout == T3_W_KN) return encode_kn_map(out, W, o.N, o.K, o.R);
    return encode_sliced_map(out, W, o.N, o.K, o.R, o.tile_n / t3::CTA_PAIR);
}

}  // namespace

struct t3_plan_s {
    uint32_t magic;
    Geometry geo;
    int device;
    int sm_count;
    float* partials;      // full partial buffers: [n_regions][R][tile_elems] fp32
    uint32_t* counters;   // [n_regions] tracker, then done[n_regions], ctl[8], status[4] (one allocation)
    uint32_t* done;
    uint32_t* ctl;
    int32_t* status;
    CUtensorMap tmX, tmW;
    float* ring;          // [ring_slots][R][tile_elems] fp32, fused mode only (NULL: fused mode uses the full buffers)
    int64_t ring_bytes;   // size of that allocation (the tuner may use fewer slots, never more)
    unsigned long long* trace;   // [trace_ctas][4] device: per-CTA timestamps of the last fused launch
    int trace_ctas;
    int last_fused_grid;  // CTAs of the last fused launch (0: none yet)
    uint32_t epoch;       // launches made so far
    t3_chunking_t user_cfg;   // the chunking as the caller gave it (zeros for NULL): the tuner's starting point
    int smem_optin;
    const void* mapX;
    const void* mapW;
    int ptr_lines_aligned;  // the cached X and W pointers are 128-byte aligned
    cudaStream_t last_stream;
    // host-pointer entry point (all lazy): two sets of device staging buffers used alternately, so that the
    // input copies of one call overlap the kernel and the output copy of the call before
    void* stageX[2];
    void* stageW[2];
    void* stageY[2];
    cudaStream_t s_in, s_out;          // plan-owned copy streams
    cudaEvent_t ev_in[2], ev_k[2], ev_out[2];   // per set: inputs landed, kernel done, output landed
    unsigned long long host_calls;
};

namespace {

bool valid(t3_plan_t p) { return p && p->magic == PLAN_MAGIC; }

// frees what the host-pointer entry point created (safe on a partly built or untouched state)
void release_host_path(t3_plan_t pl) {
    for (int b = 0; b < 2; ++b) {
        cudaFree(pl->stageX[b]); cudaFree(pl->stageW[b]); cudaFree(pl->stageY[b]);
        pl->stageX[b] = pl->stageW[b] = pl->stageY[b] = nullptr;
        if (pl->ev_in[b]) cudaEventDestroy(pl->ev_in[b]);
        if (pl->ev_k[b]) cudaEventDestroy(pl->ev_k[b]);
        if (pl->ev_out[b]) cudaEventDestroy(pl->ev_out[b]);
        pl->ev_in[b] = pl->ev_k[b] = pl->ev_out[b] = nullptr;
    }
    if (pl->s_in) cudaStreamDestroy(pl->s_in);
    if (pl->s_out) cudaStreamDestroy(pl->s_out);
    pl->s_in = pl->s_out = nullptr;
    cudaGetLastError();
}

// The fused kernel is compiled once per cluster size and reducer mode (how a region's stored tiles become Y).
typedef void (*FusedKernel)(const t3::KParams);

int reducer_mode(const t3::KParams& kp) {
    if (kp.inplace) return t3::RMODE_INPLACE;
    if (kp.partial_bf16) return t3::RMODE_BF16;
    return kp.epi.any ? t3::RMODE_RING_EPI : t3::RMODE_RING;
}

FusedKernel fused_kernel(int cluster_ctas, int rmode) {
#ifdef T3_TMA_SHARED_FETCH
    if (cluster_ctas == 4) {
        switch (rmode) {
            case t3::RMODE_RING_EPI: return t3::t3_fused_kernel<4, t3::RMODE_RING_EPI>;
            case t3::RMODE_BF16: return t3::t3_fused_kernel<4, t3::RMODE_BF16>;
            case t3::RMODE_INPLACE: return t3::t3_fused_kernel<4, t3::RMODE_INPLACE>;
            default: return t3::t3_fused_kernel<4, t3::RMODE_RING>;
        }
    }
#endif
    (void)cluster_ctas;
    switch (rmode) {
        case t3::RMODE_RING_EPI: return t3::t3_fused_kernel<2, t3::RMODE_RING_EPI>;
        case t3::RMODE_BF16: return t3::t3_fused_kernel<2, t3::RMODE_BF16>;
        case t3::RMODE_INPLACE: return t3::t3_fused_kernel<2, t3::RMODE_INPLACE>;
        default: return t3::t3_fused_kernel<2, t3::RMODE_RING>;
    }
}

int launch_kernel(const t3::KParams& kp, int cluster_ctas, int grid, int smem_bytes, cudaStream_t st) {
    fused_kernel(cluster_ctas, reducer_mode(kp))<<<grid, t3::NUM_THREADS, smem_bytes, st>>>(kp);
    return cudaGetLastError() == cudaSuccess ? T3_OK : T3_ERR_CUDA;
}

// The dynamic shared-memory attribute is per function, not per plan: always ask for the device maximum
// (for every reducer mode of this cluster size) so that plans of different sizes (and t3_gemm_rs_static)
// never lower it under one another.
// Returns the number of clusters of `cluster_ctas` CTAs that can be resident at once (0 on error).
int prepare_kernel(int cluster_ctas, int grid, int smem_optin) {
    int max_clusters = 1 << 30;
    for (int rmode = 0; rmode < 4; ++rmode) {
        const void* fn = reinterpret_cast<const void*>(fused_kernel(cluster_ctas, rmode));
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin - SMEM_STATIC_SLACK) != cudaSuccess) {
            cudaGetLastError();
            return 0;
        }
        cudaLaunchConfig_t cfg;
        std::memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
        cfg.blockDim = dim3(t3::NUM_THREADS, 1, 1);
        cfg.dynamicSmemBytes = static_cast<size_t>(smem_optin - SMEM_STATIC_SLACK);
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = static_cast<unsigned>(cluster_ctas);
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int mc = 0;
        if (cudaOccupancyMaxActiveClusters(&mc, fn, &cfg) != cudaSuccess || mc < 1) {
            cudaGetLastError();
            return 0;
        }
        if (mc < max_clusters) max_clusters = mc;
    }
    return max_clusters;
}

// Per-device ordering of t3 kernels.  The fused kernel is persistent and all of its clusters must be
// resident together, so two of them must never share the GPU.  Calls that follow each other on one stream
// are ordered by the stream itself and pay nothing; a call on a different stream than the device's
// previous t3 launch first records an event on that previous stream (which covers the launch) and makes
// its own stream wait for it - on the GPU, not on the host.
constexpr int MAX_DEVICES = 64;
struct DeviceOrder {
    std::mutex mu;
    cudaEvent_t ev = nullptr;
    cudaStream_t last_stream = nullptr;
    bool has_last = false;
};
DeviceOrder g_dev_order[MAX_DEVICES];

// RAII: holds the device's mutex for the duration of a launch sequence; enter() before the first launch,
// leave() after the last.  Inside a stream capture both do nothing (the graph orders its own nodes).
struct OrderedLaunch {
    DeviceOrder* d = nullptr;
    cudaStream_t st;
    bool capturing = false;
    OrderedLaunch(int dev, cudaStream_t s) : st(s) {
        if (dev >= 0 && dev < MAX_DEVICES) d = &g_dev_order[dev];
        if (d) d->mu.lock();
    }
    ~OrderedLaunch() {
        if (d) d->mu.unlock();
    }
    int enter() {
        if (!d) return T3_OK;
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) {
            cudaGetLastError();
            return T3_ERR_CUDA;
        }
        capturing = cs != cudaStreamCaptureStatusNone;
        if (capturing || !d->has_last || d->last_stream == st) return T3_OK;
        if (!d->ev && cudaEventCreateWithFlags(&d->ev, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            d->ev = nullptr;
            return T3_ERR_CUDA;
        }
        // the previous stream may have been destroyed since (its work then completes on its own and there
        // is nothing left to order against): a failed record is not an error of this call
        if (cudaEventRecord(d->ev, d->last_stream) != cudaSuccess) {
            cudaGetLastError();
            return T3_OK;
        }
        if (cudaStreamWaitEvent(st, d->ev, 0) != cudaSuccess) {
            cudaGetLastError();
            return T3_ERR_CUDA;
        }
        return T3_OK;
    }
    int leave() {
        if (!d || capturing) return T3_OK;
        d->last_stream = st;
        d->has_last = true;
        return T3_OK;
    }
};

t3::EpiOps make_epi(const t3_epilogue_t* e) {
    t3::EpiOps o;
    std::memset(&o, 0, sizeof o);
    if (!e) return o;
    o.bias = e->bias;
    o.residual = e->residual;
    o.keep = static_cast<const uint8_t*>(e->keep);
    o.keep_scale = e->keep_scale;
    o.bias_f32 = e->bias_dtype == T3_EPI_F32;
    o.residual_f32 = e->residual_dtype == T3_EPI_F32;
    o.any = (o.bias || o.residual || o.keep) ? 1 : 0;
    return o;
}

int check_epi(const t3_epilogue_t* e, const void* Y) {
    if (!e) return T3_OK;
    if (e->reserved != 0) return T3_ERR_INVALID_ARG;
    if ((e->bias_dtype != T3_EPI_BF16 && e->bias_dtype != T3_EPI_F32) ||
        (e->residual_dtype != T3_EPI_BF16 && e->residual_dtype != T3_EPI_F32))
        return T3_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(e->bias) | reinterpret_cast<uintptr_t>(e->residual) | reinterpret_cast<uintptr_t>(e->keep)) & 15u)
        return T3_ERR_INVALID_ARG;
    if (e->residual && e->residual == Y) return T3_ERR_INVALID_ARG;
    return T3_OK;
}

// Kernel parameters of geometry `g` over the plan's buffers.
void fill_params(t3_plan_t pl, const Geometry& g, void* Y, bool with_reduce, const t3::EpiOps& epi, t3::KParams& kp) {
    std::memset(&kp, 0, sizeof kp);
    kp.tmX = pl->tmX;
    kp.tmW = pl->tmW;
    const bool use_ring = with_reduce && pl->ring != nullptr && g.ring_slots > 0;
    kp.ring_slots = use_ring ? g.ring_slots : 0;
    kp.slot_elems = g.slot_elems;
    kp.tile_elems = g.tile_elems;
    kp.partial_bf16 = g.cfg.partial_dtype == T3_PARTIAL_BF16;
    kp.w_kn = g.cfg.w_layout == T3_W_KN;
    kp.partials = use_ring ? pl->ring : pl->partials;
    kp.Y = Y;
    kp.counters = pl->counters;
    kp.done = pl->done;
    kp.ctl = pl->ctl;
    kp.status = pl->status;
    kp.M = static_cast<int>(g.info.M);
    kp.N = static_cast<int>(g.info.N);
    kp.R = g.info.R;
    kp.chunk_rows = g.info.chunk_rows;
    kp.BN = g.info.tile_n;
    kp.sched = g.sched;
    kp.Kr = g.info.K_r;
    kp.k_align = g.k_align && pl->ptr_lines_aligned;
    kp.stages = g.info.stages;
    kp.n_acc = t3::TMEM_COLS / g.info.tile_n > t3::MAX_ACC ? t3::MAX_ACC : t3::TMEM_COLS / g.info.tile_n;
    kp.acc_stride = g.info.tile_n;
    kp.a_bytes = g.a_bytes;
    kp.b_bytes = g.b_bytes;
    kp.stage_bytes = g.stage_bytes;
    kp.gemm_ctas = g.info.gemm_ctas;
    kp.n_items = with_reduce ? g.info.n_reduce_items : 0;
    kp.red_warps = g.info.reducer_warps;
    kp.out_f32 = g.info.dtype == T3_BF16_OUT_F32;
    kp.expected = static_cast<uint32_t>(g.info.expected);
    kp.timeout_ns = static_cast<unsigned long long>(g.cfg.timeout_ms) * 1000000ull;
    kp.inplace = g.cfg.reduce == T3_REDUCE_INPLACE;
    kp.split_k = g.info.split_k;
    kp.l2_hints = g.cfg.l2_hints > 0 ? g.cfg.l2_hints : 0;
    kp.epi = epi;
    kp.trace = (with_reduce && g.info.grid <= pl->trace_ctas) ? pl->trace : nullptr;
}

int launch_fused(t3_plan_t pl, const Geometry& g, void* Y, cudaStream_t st, bool with_reduce, const t3::EpiOps& epi) {
    t3::KParams kp;
    fill_params(pl, g, Y, with_reduce, epi, kp);
    kp.epoch = ++pl->epoch;
    if (kp.epoch == 0) kp.epoch = ++pl->epoch;        // 0 is "nobody is aborting"
    if (kp.trace) pl->last_fused_grid = g.info.grid;
    return launch_kernel(kp, g.info.cluster_ctas, g.info.grid, g.info.smem_bytes, st);
}

int launch_reduce(t3_plan_t pl, const Geometry& g, void* Y, cudaStream_t st, const t3::EpiOps& epi) {
    const t3_info_t& o = g.info;
    long long blocks = (static_cast<long long>(o.n_reduce_items) + 7) / 8;      // 8 warps per block, one item each
    const long long cap = static_cast<long long>(pl->sm_count) * 8;
    if (blocks > cap) blocks = cap;
    typedef void (*ReduceKernel)(const float*, void*, int, int, int, int, int, int, t3::Sched, long long, int, t3::EpiOps);
    ReduceKernel k = epi.any ? t3::t3_reduce_kernel<t3::RMODE_RING_EPI> : t3::t3_reduce_kernel<t3::RMODE_RING>;
    if (g.cfg.reduce == T3_REDUCE_INPLACE) k = t3::t3_reduce_kernel<t3::RMODE_INPLACE>;
    else if (g.cfg.partial_dtype == T3_PARTIAL_BF16) k = t3::t3_reduce_kernel<t3::RMODE_BF16>;
    k<<<static_cast<unsigned>(blocks), 256, 0, st>>>(pl->partials, Y, static_cast<int>(o.M), static_cast<int>(o.N), o.R,
                                                     o.chunk_rows, o.dtype == T3_BF16_OUT_F32, o.tile_n, g.sched, g.slot_elems,
                                                     g.tile_elems, epi);
    return cudaGetLastError() == cudaSuccess ? T3_OK : T3_ERR_CUDA;
}

// Every cluster must be resident at once (reducers wait on tiles that other pairs produce): sets the
// kernel's shared-memory attribute and shrinks the grid to what the device can hold.
int fit_to_device(Geometry& g, int smem_optin) {
    t3_info_t& oi = g.info;
    if (oi.smem_bytes + SMEM_STATIC_SLACK > smem_optin) return T3_ERR_CUDA;
    const int cl = oi.cluster_ctas;
    const int max_clusters = prepare_kernel(cl, oi.grid, smem_optin);
    if (max_clusters < 1) return T3_ERR_CUDA;
    if (oi.grid > cl * max_clusters && g.spare_reducers > 0) {
        // the reducer-only CTAs that were added to fill idle SMs go first
        int cut = oi.grid - cl * max_clusters;
        cut = (cut + cl - 1) / cl * cl;
        if (cut > g.spare_reducers) cut = g.spare_reducers;
        g.spare_reducers -= cut;
        oi.reducer_ctas -= cut;
        oi.grid -= cut;
    }
    if (oi.grid > cl * max_clusters) {
        const int new_grid = cl * max_clusters;
        if (oi.reducer_ctas >= new_grid) return T3_ERR_UNSUPPORTED;
        oi.gemm_ctas = new_grid - oi.reducer_ctas;
        if (oi.gemm_ctas > t3::CTA_PAIR * oi.n_jobs) oi.gemm_ctas = t3::CTA_PAIR * oi.n_jobs;
        oi.grid = oi.gemm_ctas + oi.reducer_ctas;
    }
    return T3_OK;
}

// One call in `mode` with geometry `g`, ordered after the device's previous t3 launch.
int run_mode(t3_plan_t pl, const Geometry& g, int mode, void* Y, cudaStream_t st, const t3::EpiOps& epi) {
    OrderedLaunch ord(pl->device, st);
    int rc = ord.enter();
    if (rc != T3_OK) return rc;
    switch (mode) {
        case T3_MODE_FUSED: rc = launch_fused(pl, g, Y, st, true, epi); break;
        case T3_MODE_GEMM_ONLY: rc = launch_fused(pl, g, Y, st, false, epi); break;
        case T3_MODE_SEQUENTIAL:
            rc = launch_fused(pl, g, Y, st, false, epi);
            if (rc == T3_OK) rc = launch_reduce(pl, g, Y, st, epi);
            break;
        case T3_MODE_REDUCE_ONLY: rc = launch_reduce(pl, g, Y, st, epi); break;
        default: rc = T3_ERR_INVALID_ARG;
    }
    const int rc2 = ord.leave();
    return rc != T3_OK ? rc : rc2;
}

}  // namespace

extern "C" {

int t3_version(void) { return T3_VERSION; }

int t3_abi_sizes(int32_t* sizes, int32_t n) {
    const int32_t all[6] = {static_cast<int32_t>(sizeof(t3_chunking_t)), static_cast<int32_t>(sizeof(t3_info_t)),
                            static_cast<int32_t>(sizeof(t3_status_t)),   static_cast<int32_t>(sizeof(t3_epilogue_t)),
                            static_cast<int32_t>(sizeof(t3_timeline_t)), static_cast<int32_t>(sizeof(t3_tune_t))};
    for (int i = 0; sizes && i < n && i < 6; ++i) sizes[i] = all[i];
    return 6;
}
int t3_shared_fetch_available(void) { return HAVE_SHARED_FETCH ? 1 : 0; }
int t3_last_error(void) { return g_last_error; }

const char* t3_strerror(int code) {
    switch (code) {
        case T3_OK: return "ok";
        case T3_ERR_INVALID_ARG: return "invalid argument";
        case T3_ERR_SHAPE: return "unsupported shape: need M % R == 0, K % R == 0, (K/R) % 8 == 0, N % 8 == 0";
        case T3_ERR_DEVICE: return "no usable CUDA device (compute capability 10.x required)";
        case T3_ERR_ALLOC: return "device memory allocation failed";
        case T3_ERR_CUDA: return "CUDA call failed";
        case T3_ERR_TIMEOUT: return "device-side bounded wait timed out";
        case T3_ERR_UNSUPPORTED: return "unsupported option";
        case T3_ERR_TOO_LARGE: return "size beyond the supported maximum";
        default: return "unknown error";
    }
}

int t3_geometry(int64_t M, int64_t N, int64_t K, int32_t R, t3_dtype_t dtype, const t3_chunking_t* chunking,
                t3_info_t* out) {
    if (!out) return fail(T3_ERR_INVALID_ARG);
    Geometry g;
    const int rc = resolve_geometry(M, N, K, R, static_cast<int>(dtype), chunking, DEFAULT_SMS, g);
    if (rc != T3_OK) return fail(rc);
    *out = g.info;
    return T3_OK;
}

int64_t t3_schedule(int64_t M, int64_t N, int64_t K, int32_t R, t3_dtype_t dtype, const t3_chunking_t* chunking,
                    int32_t* jobs, int64_t max_jobs) {
    Geometry g;
    const int rc = resolve_geometry(M, N, K, R, static_cast<int>(dtype), chunking, DEFAULT_SMS, g);
    if (rc != T3_OK) return fail(rc);
    if (!jobs) return g.sched.n_jobs;
    if (max_jobs < g.sched.n_jobs) return fail(T3_ERR_INVALID_ARG);
    for (int j = 0; j < g.sched.n_jobs; ++j) {
        int mt, nt, r;
        t3::decode_job(g.sched, j, mt, nt, r);
        jobs[3 * j] = mt; jobs[3 * j + 1] = nt; jobs[3 * j + 2] = r;
    }
    return g.sched.n_jobs;
}

int64_t t3_reduce_schedule(int64_t M, int64_t N, int64_t K, int32_t R, t3_dtype_t dtype,
                           const t3_chunking_t* chunking, int32_t* items, int64_t max_items) {
    Geometry g;
    const int rc = resolve_geometry(M, N, K, R, static_cast<int>(dtype), chunking, DEFAULT_SMS, g);
    if (rc != T3_OK) return fail(rc);
    const int n = g.info.n_reduce_items;
    if (!items) return n;
    if (max_items < n) return fail(T3_ERR_INVALID_ARG);
    for (int t = 0; t < n; ++t) {
        const int seq = t / g.sched.items;
        int mt, nt, rb, cc, rib;
        t3::decode_region(g.sched, seq, mt, nt);
        t3::decode_item(g.sched, t % g.sched.items, rb, cc, rib);
        const int64_t row0 = static_cast<int64_t>(mt) * t3::BMJ + rb * t3::FRAG_ROWS + rib;
        const int64_t col0 = static_cast<int64_t>(nt) * g.info.tile_n + cc * t3::FRAG_COLS;
        int64_t row_end = row0 + g.sched.reduce_rows, col_end = col0 + t3::FRAG_COLS;
        if (row_end > M) row_end = M;
        if (col_end > N) col_end = N;
        if (col_end > static_cast<int64_t>(nt + 1) * g.info.tile_n) col_end = static_cast<int64_t>(nt + 1) * g.info.tile_n;
        const bool empty = row_end <= row0 || col_end <= col0;
        int32_t* it = items + 6 * static_cast<int64_t>(t);
        it[0] = mt; it[1] = nt;
        it[2] = static_cast<int32_t>(row0); it[3] = empty ? 0 : static_cast<int32_t>(row_end - row0);
        it[4] = static_cast<int32_t>(col0); it[5] = empty ? 0 : static_cast<int32_t>(col_end - col0);
    }
    return n;
}

int t3_ring_order(int32_t c, int32_t R, int32_t* order) {
    if (!order || R <= 0 || c < 0 || c >= R) return fail(T3_ERR_INVALID_ARG);
    for (int s = 0; s < R; ++s) order[s] = t3::ring_slice(c, s, R);
    return T3_OK;
}

t3_plan_t t3_plan(int64_t M, int64_t N, int64_t K, int32_t R, t3_dtype_t dtype, const t3_chunking_t* chunking) {
    int dev = 0;
    cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
        cudaGetLastError();
        fail(T3_ERR_DEVICE);
        return nullptr;
    }
    if (prop.major != 10) {
        fail(T3_ERR_DEVICE);
        return nullptr;
    }
    t3_plan_s* pl = new (std::nothrow) t3_plan_s;
    if (!pl) {
        fail(T3_ERR_ALLOC);
        return nullptr;
    }
    std::memset(static_cast<void*>(pl), 0, sizeof *pl);
    const int rc = resolve_geometry(M, N, K, R, static_cast<int>(dtype), chunking, prop.multiProcessorCount, pl->geo);
    if (rc != T3_OK) {
        delete pl;
        fail(rc);
        return nullptr;
    }
    pl->device = dev;
    pl->sm_count = prop.multiProcessorCount;
    pl->smem_optin = static_cast<int>(prop.sharedMemPerBlockOptin);
    if (chunking) pl->user_cfg = *chunking;
    const t3_info_t& o = pl->geo.info;
    {
        const int rc2 = fit_to_device(pl->geo, static_cast<int>(prop.sharedMemPerBlockOptin));
        if (rc2 != T3_OK) {
            delete pl;
            fail(rc2);
            return nullptr;
        }
    }
    const size_t pbytes = static_cast<size_t>(pl->geo.partial_bytes);
    const size_t cbytes = static_cast<size_t>(4) * (2 * o.n_regions + 64);
    if (cudaMalloc(&pl->partials, pbytes) != cudaSuccess) {
        cudaGetLastError();
        delete pl;
        fail(T3_ERR_ALLOC);
        return nullptr;
    }
    if (cudaMalloc(&pl->counters, cbytes) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(pl->partials);
        delete pl;
        fail(T3_ERR_ALLOC);
        return nullptr;
    }
    cudaMemset(pl->counters, 0, cbytes);
    if (pl->geo.ring_slots > 0) {
        const size_t rbytes = static_cast<size_t>(pl->geo.ring_slots) * pl->geo.slot_elems *
                              (pl->geo.cfg.partial_dtype == T3_PARTIAL_BF16 ? 2 : 4);
        if (cudaMalloc(&pl->ring, rbytes) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(pl->partials);
            cudaFree(pl->counters);
            delete pl;
            fail(T3_ERR_ALLOC);
            return nullptr;
        }
        pl->ring_bytes = static_cast<int64_t>(rbytes);
    }
    if (pl->geo.cfg.reduce == T3_REDUCE_INPLACE) {
        // accumulator tiles start at zero; every call's final pass leaves them at zero again
        cudaMemset(pl->partials, 0, pbytes);
        if (pl->ring) cudaMemset(pl->ring, 0, static_cast<size_t>(pl->ring_bytes));
    }
    pl->trace_ctas = pl->sm_count;
    if (cudaMalloc(&pl->trace, static_cast<size_t>(pl->trace_ctas) * 4 * sizeof(unsigned long long)) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(pl->partials);
        cudaFree(pl->counters);
        cudaFree(pl->ring);
        delete pl;
        fail(T3_ERR_ALLOC);
        return nullptr;
    }
    pl->done = pl->counters + o.n_regions;
    pl->ctl = pl->counters + 2 * o.n_regions;
    pl->status = reinterpret_cast<int32_t*>(pl->counters + 2 * o.n_regions + 8);
    pl->magic = PLAN_MAGIC;
    return pl;
}

}  // extern "C"

namespace {

// Validation, tensor maps and the launch shared by t3_gemm_rs, t3_gemm_rs_mode and t3_gemm_rs_ex.
int gemm_rs_common(t3_plan_t pl, int32_t mode, const void* X, const void* W, void* Y, const t3_epilogue_t* epi, void* stream) {
    if (!valid(pl)) return fail(T3_ERR_INVALID_ARG);
    if (mode < T3_MODE_FUSED || mode > T3_MODE_REDUCE_ONLY) return fail(T3_ERR_INVALID_ARG);
    const bool need_in = mode != T3_MODE_REDUCE_ONLY;
    const bool need_out = mode != T3_MODE_GEMM_ONLY;
    if ((need_in && (!X || !W)) || (need_out && !Y)) return fail(T3_ERR_INVALID_ARG);
    if ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(W) | reinterpret_cast<uintptr_t>(Y)) & 15u)
        return fail(T3_ERR_INVALID_ARG);
    int rc = check_epi(epi, Y);
    if (rc != T3_OK) return fail(rc);
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != pl->device) {
        cudaGetLastError();
        return fail(T3_ERR_DEVICE);
    }
    const t3_info_t& o = pl->geo.info;
    if (mode == T3_MODE_FUSED && o.reducer_warps == 0 && o.reducer_ctas == 0) return fail(T3_ERR_UNSUPPORTED);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (need_in && (X != pl->mapX || W != pl->mapW)) {
        rc = encode_sliced_map(&pl->tmX, X, o.M, o.K, o.R, t3::BM);
        if (rc == T3_OK) rc = encode_w_map(&pl->tmW, W, o);
        if (rc != T3_OK) {
            pl->mapX = pl->mapW = nullptr;
            return fail(rc);
        }
        pl->mapX = X;
        pl->mapW = W;
        pl->ptr_lines_aligned = ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(W)) & 127u) == 0;
    }
    pl->last_stream = st;
    rc = run_mode(pl, pl->geo, mode, Y, st, make_epi(epi));
    return rc == T3_OK ? T3_OK : fail(rc);
}

}  // namespace

extern "C" {

int t3_gemm_rs_mode(t3_plan_t pl, int32_t mode, const void* X, const void* W, void* Y, void* stream) {
    return gemm_rs_common(pl, mode, X, W, Y, nullptr, stream);
}

int t3_gemm_rs(t3_plan_t pl, const void* X, const void* W, void* Y, void* stream) {
    if (!valid(pl)) return fail(T3_ERR_INVALID_ARG);
    return gemm_rs_common(pl, pl->geo.cfg.mode, X, W, Y, nullptr, stream);
}

int t3_gemm_rs_ex(t3_plan_t pl, const void* X, const void* W, void* Y, const t3_epilogue_t* epi, void* stream) {
    if (!valid(pl)) return fail(T3_ERR_INVALID_ARG);
    return gemm_rs_common(pl, pl->geo.cfg.mode, X, W, Y, epi, stream);
}

int t3_gemm_rs_host(t3_plan_t pl, const void* Xh, const void* Wh, void* Yh, void* stream) {
    if (!valid(pl) || !Xh || !Wh || !Yh) return fail(T3_ERR_INVALID_ARG);
    const t3_info_t& o = pl->geo.info;
    const size_t xb = static_cast<size_t>(2) * o.M * o.K, wb = static_cast<size_t>(2) * o.K * o.N;
    const size_t yb = static_cast<size_t>(o.dtype == T3_BF16_OUT_F32 ? 4 : 2) * o.M * o.N;
    if (!pl->stageX[0]) {
        bool ok = cudaStreamCreateWithFlags(&pl->s_in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&pl->s_out, cudaStreamNonBlocking) == cudaSuccess;
        for (int b = 0; ok && b < 2; ++b)
            ok = cudaMalloc(&pl->stageX[b], xb) == cudaSuccess && cudaMalloc(&pl->stageW[b], wb) == cudaSuccess &&
                 cudaMalloc(&pl->stageY[b], yb) == cudaSuccess &&
                 cudaEventCreateWithFlags(&pl->ev_in[b], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&pl->ev_k[b], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&pl->ev_out[b], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) {
            cudaGetLastError();
            release_host_path(pl);
            return fail(T3_ERR_ALLOC);
        }
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int b = static_cast<int>(pl->host_calls & 1ull);
    // inputs of this call -> set b, as soon as the kernel that last read set b (two calls ago) is done
    // (an event that was never recorded does not block)
    bool ok = cudaStreamWaitEvent(pl->s_in, pl->ev_k[b], 0) == cudaSuccess &&
              cudaMemcpyAsync(pl->stageX[b], Xh, xb, cudaMemcpyHostToDevice, pl->s_in) == cudaSuccess &&
              cudaMemcpyAsync(pl->stageW[b], Wh, wb, cudaMemcpyHostToDevice, pl->s_in) == cudaSuccess &&
              cudaEventRecord(pl->ev_in[b], pl->s_in) == cudaSuccess &&
              // the kernel, on the caller's stream: after its inputs landed and set b's previous output left
              cudaStreamWaitEvent(st, pl->ev_in[b], 0) == cudaSuccess &&
              cudaStreamWaitEvent(st, pl->ev_out[b], 0) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        return fail(T3_ERR_CUDA);
    }
    const int rc = t3_gemm_rs_mode(pl, pl->geo.cfg.mode, pl->stageX[b], pl->stageW[b], pl->stageY[b], stream);
    if (rc != T3_OK) return rc;
    // the result, on the output stream; the caller's stream then waits for it, so that everything the caller
    // enqueues after this call (or a synchronisation of `stream`) sees Y_host complete
    ok = cudaEventRecord(pl->ev_k[b], st) == cudaSuccess &&
         cudaStreamWaitEvent(pl->s_out, pl->ev_k[b], 0) == cudaSuccess &&
         cudaMemcpyAsync(Yh, pl->stageY[b], yb, cudaMemcpyDeviceToHost, pl->s_out) == cudaSuccess &&
         cudaEventRecord(pl->ev_out[b], pl->s_out) == cudaSuccess &&
         cudaStreamWaitEvent(st, pl->ev_out[b], 0) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        return fail(T3_ERR_CUDA);
    }
    ++pl->host_calls;
    return T3_OK;
}

int t3_plan_info(t3_plan_t pl, t3_info_t* out) {
    if (!valid(pl) || !out) return fail(T3_ERR_INVALID_ARG);
    *out = pl->geo.info;
    return T3_OK;
}

int t3_plan_partials(t3_plan_t pl, void** partials, int64_t* bytes) {
    if (!valid(pl) || !partials) return fail(T3_ERR_INVALID_ARG);
    *partials = pl->partials;
    if (bytes) *bytes = pl->geo.partial_bytes;
    return T3_OK;
}

int t3_plan_ring(t3_plan_t pl, void** ring, int64_t* bytes) {
    if (!valid(pl) || !ring) return fail(T3_ERR_INVALID_ARG);
    *ring = pl->ring;
    if (bytes) *bytes = pl->ring ? pl->ring_bytes : 0;
    return T3_OK;
}

int t3_plan_timeline(t3_plan_t pl, t3_timeline_t* out) {
    if (!valid(pl) || !out) return fail(T3_ERR_INVALID_ARG);
    std::memset(out, 0, sizeof *out);
    if (pl->last_fused_grid <= 0) return fail(T3_ERR_UNSUPPORTED);       // no fused call yet
    if (cudaStreamSynchronize(pl->last_stream) != cudaSuccess) {
        cudaGetLastError();
        return fail(T3_ERR_CUDA);
    }
    const int n = pl->last_fused_grid;
    unsigned long long h[4 * 160];
    if (n > 160 || cudaMemcpy(h, pl->trace, static_cast<size_t>(n) * 4 * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return fail(T3_ERR_CUDA);
    }
    unsigned long long t0 = ~0ull, t_pub = 0, t_red = 0, t_end = 0;
    for (int i = 0; i < n; ++i) {
        t0 = std::min(t0, h[4 * i]);
        t_pub = std::max(t_pub, h[4 * i + 1]);
        t_red = std::max(t_red, h[4 * i + 2]);
        t_end = std::max(t_end, h[4 * i + 3]);
    }
    if (t_pub < t0) t_pub = t0;
    if (t_red < t_pub) t_red = t_pub;
    if (t_end < t_red) t_end = t_red;
    out->total_us = 1e-3 * static_cast<double>(t_end - t0);
    out->produce_us = 1e-3 * static_cast<double>(t_pub - t0);
    out->tail_us = 1e-3 * static_cast<double>(t_red - t_pub);
    out->drain_us = 1e-3 * static_cast<double>(t_end - t_red);
    out->ctas = n;
    return T3_OK;
}

int t3_plan_export_partials(t3_plan_t pl, void* dst, void* stream) {
    if (!valid(pl) || !dst || (reinterpret_cast<uintptr_t>(dst) & 3u)) return fail(T3_ERR_INVALID_ARG);
    if (pl->geo.cfg.reduce == T3_REDUCE_INPLACE) return fail(T3_ERR_UNSUPPORTED);
    const Geometry& g = pl->geo;
    const t3_info_t& o = g.info;
    const long long total = static_cast<long long>(o.R) * o.M * o.N;
    long long blocks = (total + 255) / 256;
    const long long cap = static_cast<long long>(pl->sm_count) * 16;
    if (blocks > cap) blocks = cap;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    t3::t3_export_partials_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(
        pl->partials, static_cast<float*>(dst), static_cast<int>(o.M), static_cast<int>(o.N), o.R, o.tile_n, g.sched,
        g.slot_elems, g.tile_elems, g.cfg.partial_dtype == T3_PARTIAL_BF16);
    pl->last_stream = st;
    return cudaGetLastError() == cudaSuccess ? T3_OK : fail(T3_ERR_CUDA);
}

int t3_plan_status(t3_plan_t pl, t3_status_t* out) {
    if (!valid(pl)) return fail(T3_ERR_INVALID_ARG);
    if (cudaStreamSynchronize(pl->last_stream) != cudaSuccess) {
        cudaGetLastError();
        return fail(T3_ERR_CUDA);
    }
    int32_t h[4] = {0, 0, 0, 0};
    if (cudaMemcpy(h, pl->status, sizeof h, cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return fail(T3_ERR_CUDA);
    }
    if (out) {
        out->code = h[0]; out->where = h[1]; out->block = h[2]; out->detail = h[3];
    }
    if (h[0] != 0) {
        // a wait ran out: the kernel has returned; clear the status word (the kernel's last CTA
        // has already re-armed the tracker counters)
        cudaMemset(pl->status, 0, sizeof h);
        cudaMemset(pl->counters, 0, static_cast<size_t>(4) * (2 * pl->geo.info.n_regions + 8));
        if (pl->geo.cfg.reduce == T3_REDUCE_INPLACE) {
            // half-accumulated tiles of the aborted call
            cudaMemset(pl->partials, 0, static_cast<size_t>(pl->geo.partial_bytes));
            if (pl->ring) cudaMemset(pl->ring, 0, static_cast<size_t>(pl->ring_bytes));
        }
        return fail(h[0]);
    }
    return T3_OK;
}

// ---------------------------------------------------------------------------------------------
// t3_gemm_rs_static: scratch in a file-scope device array, no allocation of any kind.
// In host code the array's name is only a handle for cudaGetSymbolAddress, never a device address.
// ---------------------------------------------------------------------------------------------
}  // extern "C"

namespace {

static __device__ __align__(256) unsigned char g_static_scratch[T3_STATIC_SCRATCH_BYTES];

constexpr int MAX_STATIC_DEVICES = 64;
struct StaticDeviceState {
    int ready;            // 0 = not set up, 1 = ok, negative = the error the set-up hit
    void* scratch;        // device address of g_static_scratch on this device
    int sm_count;
    int cc_major;
    int max_clusters;     // resident CTA pairs of the fused kernel at its largest shared-memory size
    int smem_optin;       // opt-in shared memory per block
};
StaticDeviceState g_static_dev[MAX_STATIC_DEVICES];   // zero-initialised; written once per device
std::once_flag g_static_once[MAX_STATIC_DEVICES];

// Once per device, with that device current; host threads making their first calls together meet in
// std::call_once, so each sees the fields complete.
int static_device_setup(int dev, StaticDeviceState** out) {
    if (dev < 0 || dev >= MAX_STATIC_DEVICES) return T3_ERR_DEVICE;
    StaticDeviceState& st = g_static_dev[dev];
    std::call_once(g_static_once[dev], [&st, dev]() {
        int rc = 1;
        void* ptr = nullptr;
        int sms = 0, major = 0, smem_optin = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
            cudaGetLastError();
            rc = T3_ERR_DEVICE;
        } else if (major != 10) {
            rc = T3_ERR_DEVICE;
        } else if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            rc = T3_ERR_CUDA;
        } else {
            const int mc = prepare_kernel(t3::CTA_PAIR, sms & ~1, smem_optin);
            if (mc < 1) {
                rc = T3_ERR_CUDA;
            } else {
                st.scratch = ptr;
                st.sm_count = sms;
                st.cc_major = major;
                st.max_clusters = mc;
                st.smem_optin = smem_optin;
            }
        }
        st.ready = rc;
    });
    if (st.ready != 1) return st.ready;
    *out = &st;
    return T3_OK;
}

}  // namespace

extern "C" {

int t3_gemm_rs_static(int64_t M, int64_t N, int64_t K, int32_t R, t3_dtype_t dtype, const void* X, const void* W,
                      void* Y, void* stream) {
    if (!X || !W || !Y) return fail(T3_ERR_INVALID_ARG);
    if ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(W) | reinterpret_cast<uintptr_t>(Y)) & 15u)
        return fail(T3_ERR_INVALID_ARG);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return fail(T3_ERR_DEVICE);
    }
    StaticDeviceState* st = nullptr;
    int rc = static_device_setup(dev, &st);
    if (rc != T3_OK) return fail(rc);

    t3_chunking_t ch;
    std::memset(&ch, 0, sizeof ch);
    ch.mode = T3_MODE_FUSED;
    ch.ring_slots = -1;                       // partial tiles in full buffers, inside the static array
    ch.cluster_ctas = t3::CTA_PAIR;
    ch.l2_hints = -1;
    Geometry g;                               // on the stack: no heap either
    rc = resolve_geometry(M, N, K, R, static_cast<int>(dtype), &ch, st->sm_count, g);
    if (rc != T3_OK) return fail(rc);
    t3_info_t& o = g.info;
    if (o.smem_bytes + SMEM_STATIC_SLACK > st->smem_optin) return fail(T3_ERR_CUDA);
    if (o.grid > t3::CTA_PAIR * st->max_clusters) {          // every pair must be resident at once
        o.gemm_ctas = t3::CTA_PAIR * st->max_clusters;
        if (o.gemm_ctas > t3::CTA_PAIR * o.n_jobs) o.gemm_ctas = t3::CTA_PAIR * o.n_jobs;
        o.grid = o.gemm_ctas;
    }
    // layout of the static array: [partial tiles, rounded up to 256][counters | done | ctl | status]
    const unsigned long long pbytes = (static_cast<unsigned long long>(g.partial_bytes) + 255ull) & ~255ull;
    const unsigned long long tbytes = 4ull * (2ull * o.n_regions + 64ull);
    if (pbytes + tbytes > static_cast<unsigned long long>(T3_STATIC_SCRATCH_BYTES)) return fail(T3_ERR_TOO_LARGE);
    unsigned char* base = static_cast<unsigned char*>(st->scratch);
    uint32_t* tracker = reinterpret_cast<uint32_t*>(base + pbytes);

    t3::KParams kp;
    std::memset(&kp, 0, sizeof kp);
    rc = encode_sliced_map(&kp.tmX, X, M, K, R, t3::BM);
    if (rc == T3_OK) rc = encode_w_map(&kp.tmW, W, o);
    if (rc != T3_OK) return fail(rc);
    kp.partials = reinterpret_cast<float*>(base);
    kp.ring_slots = 0;
    kp.slot_elems = g.slot_elems;
    kp.tile_elems = g.tile_elems;
    kp.Y = Y;
    kp.counters = tracker;
    kp.done = tracker + o.n_regions;
    kp.ctl = tracker + 2 * o.n_regions;
    kp.status = reinterpret_cast<int32_t*>(tracker + 2 * o.n_regions + 8);
    kp.M = static_cast<int>(M);
    kp.N = static_cast<int>(N);
    kp.R = R;
    kp.chunk_rows = o.chunk_rows;
    kp.BN = o.tile_n;
    kp.sched = g.sched;
    kp.Kr = o.K_r;
    kp.k_align = g.k_align && ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(W)) & 127u) == 0;
    kp.stages = o.stages;
    kp.n_acc = t3::TMEM_COLS / o.tile_n > t3::MAX_ACC ? t3::MAX_ACC : t3::TMEM_COLS / o.tile_n;
    kp.acc_stride = o.tile_n;
    kp.a_bytes = g.a_bytes;
    kp.b_bytes = g.b_bytes;
    kp.stage_bytes = g.stage_bytes;
    kp.gemm_ctas = o.gemm_ctas;
    kp.n_items = o.n_reduce_items;
    kp.red_warps = o.reducer_warps;
    kp.out_f32 = dtype == T3_BF16_OUT_F32;
    kp.expected = static_cast<uint32_t>(o.expected);
    kp.timeout_ns = static_cast<unsigned long long>(g.cfg.timeout_ms) * 1000000ull;
    kp.split_k = 1;
    kp.epoch = 1;             // the tracker words, ctl[2] among them, are cleared before every launch

    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left: the tracker must start at zero
    if (cudaMemsetAsync(tracker, 0, static_cast<size_t>(tbytes), cs) != cudaSuccess) {
        cudaGetLastError();
        return fail(T3_ERR_CUDA);
    }
    if (launch_kernel(kp, t3::CTA_PAIR, o.grid, o.smem_bytes, cs) != T3_OK) return fail(T3_ERR_CUDA);
    return T3_OK;
}

int t3_plan_tune(t3_plan_t pl, const void* X, const void* W, void* Y, void* stream, t3_tune_t* out) {
    if (!valid(pl) || !X || !W || !Y) return fail(T3_ERR_INVALID_ARG);
    if (out) std::memset(out, 0, sizeof *out);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    {
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(st, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) {
            cudaGetLastError();
            return fail(T3_ERR_UNSUPPORTED);
        }
    }
    if (pl->geo.cfg.mode != T3_MODE_FUSED) return T3_OK;        // the caller fixed the mode: nothing to choose
    // a first ordinary call: validates the pointers and the device, encodes the tensor maps
    int rc = gemm_rs_common(pl, T3_MODE_FUSED, X, W, Y, nullptr, stream);
    if (rc != T3_OK) return rc;
    t3_status_t stt;
    rc = t3_plan_status(pl, &stt);
    if (rc != T3_OK) return rc;

    const Geometry cur = pl->geo;
    const t3_info_t& o = cur.info;
    const int esize = cur.cfg.partial_dtype == T3_PARTIAL_BF16 ? 2 : 4;
    const int64_t slot_bytes = cur.slot_elems * esize;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        cudaGetLastError();
        if (e0) cudaEventDestroy(e0);
        return fail(T3_ERR_CUDA);
    }
    constexpr int MAX_CAND = 48, TIMED = 5;
    // the plan's own full partial buffers double as the buffer whose rewrite sweeps the L2 between timed
    // calls: every mode rewrites them before reading them (update in place: they hold zeros between calls)
    const size_t flush_bytes = std::min(static_cast<size_t>(cur.partial_bytes), static_cast<size_t>(512) << 20);
    Geometry best = cur;
    float best_us = 0.f, cur_us = 0.f;
    int n = 0, chosen = 0;
    const int kinds[3] = {0, 1, 2};                 // fused + ring, fused + full buffers, sequential
    const int rrs[2] = {cur.cfg.reduce_rows, cur.cfg.reduce_rows == 32 ? 16 : 32};
    const int cls[2] = {o.cluster_ctas, o.cluster_ctas == 2 ? 4 : 2};
    const int gts[2] = {o.group_tiles, o.group_tiles / 2};
    const t3::EpiOps no_epi = make_epi(nullptr);
    // median of TIMED calls of geometry g in mode `mode`, each after an L2 sweep; negative on failure
    auto time_config = [&](const Geometry& g, int mode) -> float {
        float us[TIMED];
        bool ok = run_mode(pl, g, mode, Y, st, no_epi) == T3_OK;
        for (int t = 0; ok && t < TIMED; ++t) {
            ok = cudaMemsetAsync(pl->partials, 0, flush_bytes, st) == cudaSuccess &&
                 cudaEventRecord(e0, st) == cudaSuccess && run_mode(pl, g, mode, Y, st, no_epi) == T3_OK &&
                 cudaEventRecord(e1, st) == cudaSuccess && cudaEventSynchronize(e1) == cudaSuccess;
            float ms = 0.f;
            ok = ok && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess;
            us[t] = 1e3f * ms;
        }
        pl->last_stream = st;
        t3_status_t s2;
        if (!ok || t3_plan_status(pl, &s2) != T3_OK) {
            cudaGetLastError();
            return -1.f;
        }
        std::sort(us, us + TIMED);
        return us[TIMED / 2];
    };
    // bring the clocks up before the first candidate is timed: at least three calls and ~20 ms of work
    {
        const float first = time_config(cur, cur.cfg.mode);
        const int more = first > 0.f ? static_cast<int>(20000.f / first) : 0;
        for (int i = 0; i < more && i < 200; ++i) run_mode(pl, cur, cur.cfg.mode, Y, st, no_epi);
    }
    for (int ki = 0; ki < 3; ++ki)
        for (int ri = 0; ri < 2; ++ri)
            for (int ci = 0; ci < 2; ++ci)
                for (int gi = 0; gi < 2; ++gi) {
                    if (n >= MAX_CAND) break;
                    if (gts[gi] < 1 || (gi == 1 && gts[1] == gts[0])) continue;
                    t3_chunking_t c = pl->user_cfg;
                    c.tile_n = o.tile_n;                      // the workspace is laid out for this tile width
                    c.mode = kinds[ki] == 2 ? T3_MODE_SEQUENTIAL : T3_MODE_FUSED;
                    c.reduce_rows = rrs[ri];
                    c.cluster_ctas = cls[ci];
                    c.group_tiles = gts[gi];
                    if (kinds[ki] == 0) {
                        if (!pl->ring) continue;
                        c.ring_slots = pl->user_cfg.ring_slots > 0 ? pl->user_cfg.ring_slots : 0;
                    } else {
                        c.ring_slots = -1;
                    }
                    Geometry g;
                    if (resolve_geometry(o.M, o.N, o.K, o.R, o.dtype, &c, pl->sm_count, g) != T3_OK) continue;
                    if (kinds[ki] == 0) {
                        if (g.ring_slots == 0) continue;      // resolves to full buffers: same as kind 1
                        if (g.ring_slots * slot_bytes > pl->ring_bytes) {
                            c.ring_slots = static_cast<int32_t>(pl->ring_bytes / slot_bytes);   // what is allocated
                            if (c.ring_slots < c.group_tiles ||
                                resolve_geometry(o.M, o.N, o.K, o.R, o.dtype, &c, pl->sm_count, g) != T3_OK || g.ring_slots == 0)
                                continue;
                        }
                    }
                    if (g.info.tile_n != o.tile_n || g.partial_bytes != cur.partial_bytes) continue;
                    if (fit_to_device(g, pl->smem_optin) != T3_OK) continue;
                    // one untimed call, then TIMED timed ones, each after the L2 has been swept (a sublayer's
                    // operands are cold when it runs inside a model: other layers' weights have passed through
                    // the cache since its last call)
                    const float med = time_config(g, c.mode);
                    if (med <= 0.f) continue;
                    if (out) {
                        out->mode[n] = c.mode; out->ring_slots[n] = g.ring_slots; out->reduce_rows[n] = g.info.reduce_rows;
                        out->cluster_ctas[n] = g.info.cluster_ctas; out->group_tiles[n] = g.info.group_tiles; out->us[n] = med;
                    }
                    if (n == 0) cur_us = med;                 // the first candidate is the current configuration
                    if (n == 0 || med < best_us) {
                        best_us = med;
                        best = g;
                        chosen = n;
                    }
                    ++n;
                }
    if (n > 0 && chosen != 0) {
        // the current configuration once more, now that everything else has run: drift of the GPU's power
        // state over the trial must not pass for a better candidate
        const float again = time_config(cur, cur.cfg.mode);
        if (again > 0.f && again < cur_us) cur_us = again;
        if (out) out->us[0] = cur_us;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (n == 0) return fail(T3_ERR_CUDA);
    // keep the current configuration unless the best candidate is at least 3 % faster (5 % when that means
    // giving up the fused mode for the sequential one: on multi-millisecond shapes the power state alone moves
    // a measurement by 3 %)
    const float need = best.cfg.mode != cur.cfg.mode ? 0.95f : 0.97f;
    if (chosen != 0 && best_us > need * cur_us) {
        best = cur;
        chosen = 0;
    }
    pl->geo = best;
    pl->geo.info.tuned = 1;
    pl->geo.info.mode = pl->geo.cfg.mode;
    if (out) {
        out->n_tried = n;
        out->chosen = chosen;
    }
    // leave Y written by the chosen configuration
    return gemm_rs_common(pl, pl->geo.cfg.mode, X, W, Y, nullptr, stream);
}

int t3_destroy(t3_plan_t pl) {
    if (!pl) return T3_OK;
    if (!valid(pl)) return fail(T3_ERR_INVALID_ARG);
    cudaDeviceSynchronize();
    cudaGetLastError();
    cudaFree(pl->partials);
    cudaFree(pl->ring);
    cudaFree(pl->counters);
    cudaFree(pl->trace);
    release_host_path(pl);
    pl->magic = 0;
    delete pl;
    return T3_OK;
}

}  // extern "C"
