// Producer-tile and reducer-ticket order, shared by host (plan, queries) and device.
//
// A producer job is one BMJ x BN output tile of one K-slice, computed by a CTA
// pair (cta_group::2: each CTA owns BM = 128 of the BMJ = 256 rows and supplies
// half of the B operand).  Each output tile is produced R times (once per
// slice) and is also the tracker's region (paper Section 4.2.1: one counter per
// producer tile, threshold = tile size x updates per element; here the unit is
// one CTA's 128-row half of a partial tile, so threshold = 2 * R).
//
// n_mt counts BMJ-row blocks, G is the group height in such blocks.
//
// Order (the single-GPU analog of Section 4.4's staggered scheduling: the order
// decides when a region's trigger can fire).  Default ("grouped"): row tiles
// are taken in groups of G; inside a group the order is
// n_tile -> slice -> row tile  (row tile fastest), so the R partials of one
// output tile are produced within G*R consecutive jobs, a W_r tile is reused
// by G consecutive jobs, and a region completes - and its reduction starts -
// long before the GEMM ends.
//
// For study, the paper's own staggered order (Section 4.4) is available too:
// R steps; in step s the simulated device r produces the chunk (r + s + 1) mod R,
// its own chunk last, so that in a real ring every step's output is what the
// next device needs next.  On one GPU every region then completes only during
// the last step.
#pragma once
#include <cstdint>

#if defined(__CUDACC__)
#define T3_HD __host__ __device__ __forceinline__
#else
#define T3_HD inline
#endif

namespace t3 {

constexpr int BM = 128;   // rows per CTA (one 128-lane TMEM accumulator)
constexpr int CTA_PAIR = 2;
constexpr int BMJ = BM * CTA_PAIR;   // rows of a producer job / tracker region
constexpr int BK = 64;    // bf16 elements per k-block = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int EPI_WARPS = 4;

// Partial-tile storage ("fragment-major").  A BMJ x BN partial tile is kept as 8 row blocks (32 rows:
// the rows one epilogue warp drains) x nc column chunks (32 columns) of 1024 floats.  Inside a chunk
// the floats are ordered exactly as the epilogue lanes hold them after the 16x256b TMEM load, so that
// every epilogue store instruction and every reducer load instruction covers 512 contiguous bytes
// (four full 128-byte lines):
//   float index = ((rowsel * 2 + jp) * 32 + lane) * 4 + e,    lane = 4 * g + q
//   row in block = g + 8 * rowsel                             (g 0..7, rowsel 0..3)
//   col in chunk = 16 * jp + 8 * (e >> 1) + 2 * q + (e & 1)   (jp 0..1, q 0..3, e 0..3)
// A float4 therefore holds two pairs of neighbouring columns of one row; the reducer regroups the
// sums among the four lanes of a row before it writes Y.
// With 16-bit partial tiles (the "wire" type of Section 5.2) a chunk is 1024 bf16 and a lane's eight
// values of one row (jp = 0 and 1) are stored together as 16 bytes:
//   bf16 index = ((rowsel * 32 + lane) * 8 + jp * 4 + e
// so a chunk is written with four and read with four 128-bit accesses per lane.
constexpr int FRAG_ROWS = 32;
constexpr int FRAG_COLS = 32;
constexpr int FRAG_ELEMS = FRAG_ROWS * FRAG_COLS;
constexpr int ROW_BLOCKS = BMJ / FRAG_ROWS;   // 8

// element offset of (row, col) of a tile (row < BMJ, col < 32 * nc) inside the tile's storage
T3_HD int64_t frag_offset(int row, int col, int nc, bool bf16 = false) {
    const int rb = row / FRAG_ROWS, rr = row % FRAG_ROWS;
    const int cc = col / FRAG_COLS, c = col % FRAG_COLS;
    const int g = rr & 7, rowsel = rr >> 3;
    const int jp = c >> 4, c16 = c & 15;
    const int e = ((c16 >> 3) << 1) | (c16 & 1), q = (c16 & 7) >> 1;
    const int64_t chunk = (static_cast<int64_t>(rb) * nc + cc) * FRAG_ELEMS;
    if (bf16) return chunk + (rowsel * 32 + (4 * g + q)) * 8 + jp * 4 + e;
    return chunk + ((rowsel * 2 + jp) * 32 + (4 * g + q)) * 4 + e;
}

struct Sched {
    int n_mt, n_nt, R, G;
    int full_group_jobs;      // G * n_nt * R
    int full_group_regions;   // G * n_nt
    int n_jobs, n_regions;
    int nc;                   // 32-column chunks per tile = ceil(BN / 32)
    int reduce_rows;          // rows of a reducer item: 32 (a whole chunk) or 16 (half of one)
    int items;                // reducer items per region = 8 row blocks x nc chunks x (32 / reduce_rows)
    int staggered;            // 1: the paper's staggered order (needs whole tiles per chunk)
    int tpc;                  // staggered: row tiles per reduce-scatter chunk
};

T3_HD Sched make_sched(int n_mt, int n_nt, int R, int G, int reduce_rows, int BN) {
    Sched s;
    s.n_mt = n_mt; s.n_nt = n_nt; s.R = R; s.G = G;
    s.full_group_jobs = G * n_nt * R;
    s.full_group_regions = G * n_nt;
    s.n_jobs = n_mt * n_nt * R;
    s.n_regions = n_mt * n_nt;
    s.nc = (BN + FRAG_COLS - 1) / FRAG_COLS;
    s.reduce_rows = reduce_rows;
    s.items = ROW_BLOCKS * s.nc * (FRAG_ROWS / reduce_rows);
    s.staggered = 0;
    s.tpc = 0;
    return s;
}

// job j -> (row block of BMJ rows, column tile, slice)
// seq: the region's sequence number in completion order (inverse of decode_region)
T3_HD void decode_job(const Sched& s, int j, int& mt, int& nt, int& r, int& seq) {
    if (s.staggered) {
        // step -> device -> row tile of the device's chunk of that step -> column tile
        const int per_dev = s.tpc * s.n_nt;
        const int step = j / (s.R * per_dev);
        const int rem = j - step * s.R * per_dev;
        r = rem / per_dev;
        const int rem2 = rem - r * per_dev;
        const int ti = rem2 / s.n_nt;
        nt = rem2 - ti * s.n_nt;
        mt = ((r + step + 1) % s.R) * s.tpc + ti;
        seq = mt * s.n_nt + nt;          // regions complete in the last step, in this order
        return;
    }
    const int g = j / s.full_group_jobs;
    const int rem = j - g * s.full_group_jobs;
    const int left = s.n_mt - g * s.G;
    const int Gg = left < s.G ? left : s.G;
    const int mi = rem % Gg;
    const int q = rem / Gg;
    r = q % s.R;
    nt = q / s.R;
    mt = g * s.G + mi;
    seq = g * s.full_group_regions + nt * Gg + mi;
}
T3_HD void decode_job(const Sched& s, int j, int& mt, int& nt, int& r) {
    int seq;
    decode_job(s, j, mt, nt, r, seq);
}

// region sequence number (completion order) -> (row tile, column tile)
T3_HD void decode_region(const Sched& s, int seq, int& mt, int& nt) {
    if (s.staggered) {
        mt = seq / s.n_nt;
        nt = seq - mt * s.n_nt;
        return;
    }
    const int g = seq / s.full_group_regions;
    const int rem = seq - g * s.full_group_regions;
    const int left = s.n_mt - g * s.G;
    const int Gg = left < s.G ? left : s.G;
    mt = g * s.G + rem % Gg;
    nt = rem / Gg;
}

// reducer item `it` of a region (0 <= it < items per region) -> row block, column chunk, first row inside the block;
// halves of a chunk are neighbours, chunks of a row block follow each other
T3_HD void decode_item(const Sched& s, int it, int& rb, int& cc, int& row_in_block) {
    const int halves = FRAG_ROWS / s.reduce_rows;
    const int h = it % halves;
    const int ch = it / halves;
    cc = ch % s.nc;
    rb = ch / s.nc;
    row_in_block = h * s.reduce_rows;
}

// Ring order of chunk c (Section 4.1 four-device example): the s-th partial
// added is the one of device (c - 1 - s) mod R; the owner's own comes last.
T3_HD int ring_slice(int c, int s, int R) {
    int d = (c - 1 - s) % R;
    return d < 0 ? d + R : d;
}

}  // namespace t3
