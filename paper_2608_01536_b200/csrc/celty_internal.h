// Internal definitions shared by the host encoder and the CUDA translation unit.
#pragma once
#include <cstddef>
#include <cstdint>
#include <vector>

#include "celty.h"

namespace celty {

constexpr int kGroup = 8;            // entries per 16-byte value vector / 32-bit run word
constexpr int kChunkGroups = 32;     // COLUMN layout: groups per warp-wide chunk (256 entries)
constexpr int kTileSlack = 8;        // LANE_TILE: spare accumulator rows per slab for group-tail slots
// LANE_TILE sub-block header (bytes), ahead of the value vectors and run words:
//   [0,32)   groups of 8 entries that lane L's tile holds (u8)
//   [32,36)  vectors in the sub-block | steps << 16 (u32), steps = the largest group count;  rest zero
constexpr int kSubHeader = 48;
constexpr int kMaxTileRows = 240;    // keeps local rows (and the spare rows after them) in a byte
constexpr int64_t kMaxM = 49152;     // accumulators of one thread block must fit shared memory
constexpr size_t kAlign = 256;
constexpr int kMaxBlocks = 192;      // blocks of the fused kernel the workspace has partial vectors for
// LANE_TILE: a thread block covers at most this many slabs of rows.  The kernels take any value; with one
// slab per block (row parts = slabs, all of a block's warp teams work on different columns of the same rows)
// every configured shape ran as fast or faster on B200 than with 2 or 4, mostly because a block then adds
// fewer rows into y at the end.
constexpr int kSlabsPerBlock = 1;

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

#ifdef __CUDACC__
#define CELTY_HD __host__ __device__
#else
#define CELTY_HD
#endif

// LANE_TILE row map.  Rows are dealt to the 32 lanes one at a time (row r belongs to lane r mod 32), and
// the groups of 32 consecutive rows are dealt to the S slabs in chunks of C groups, round robin.  Tile
// t = 32*s + L is the ordered set of rows that lane L of slab s receives; local row i of that tile is
//     row = (((i / C) * S + s) * C + i mod C) * 32 + L.
// A lane's local rows grow with the row number, every slab samples the whole height of the matrix (so a
// mask whose density drifts with the row index still gives every lane and every slab the same share),
// and local rows [kC, kC + C) of a slab are the 32*C consecutive rows that start at ((k*S + s)*C)*32:
// the accumulator word (i*32 + L) order of a slab is the order of y, C*32 rows at a time.
CELTY_HD inline int64_t tile_row(int64_t S, int64_t C, int64_t s, int64_t lane, int64_t i)
{
    return (((i / C) * S + s) * C + i % C) * 32 + lane;
}

// Workspace layout (device): all offsets multiples of 256.
struct WorkspaceLayout {
    size_t status_off;   // uint32 status, int32 count, uint32 tickets[2] (and spare words)
    size_t idx_off;      // int32[K]
    size_t val_off;      // uint16[K]
    size_t scratch_off;  // uint32[T + 2] for celty_decode_device
    size_t partial_off;  // float[kMaxBlocks][part_words]: per-block partial sums of the fused kernel
    size_t total;
};

inline WorkspaceLayout workspace_layout(int64_t K, int64_t T, int64_t part_words)
{
    WorkspaceLayout w{};
    w.status_off = 0;
    w.idx_off = kAlign;
    w.val_off = w.idx_off + round_up((size_t)K * 4, kAlign);
    w.scratch_off = w.val_off + round_up((size_t)K * 2, kAlign);
    w.partial_off = w.scratch_off + round_up((size_t)(T + 2) * 4, kAlign);
    w.total = w.partial_off + round_up((size_t)kMaxBlocks * part_words * 4, kAlign);
    return w;
}

}  // namespace celty

// The handle.  Host side: logical block pointers and the packed image exactly as it is copied to
// the device.  Device side: caller-owned buffers recorded by celty_bind_device.
struct celty_matrix {
    int64_t M = 0, K = 0;
    int32_t layout = 0;
    int32_t R = 0;          // local rows per tile (LANE_TILE) or M (COLUMN)
    int32_t C = 1;          // LANE_TILE: groups of 32 rows that go to the same slab in a row (see tile_row)
    int64_t T = 1;          // tiles per column (LANE_TILE: 32 * S)
    int64_t S = 1;          // slabs of 32 tiles per column (LANE_TILE), 1 for COLUMN
    int32_t P = 1, Sc = 1;  // LANE_TILE: row parts per column and slabs per part (P * Sc >= S)
    int64_t nnz = 0, n_pad = 0;
    std::vector<uint32_t> block_ptr;   // K*T + 1, stored entries before block (j, t)
    std::vector<uint8_t> pad_bits;     // one bit per stored entry (logical order): 1 = padding entry
    // image = [meta | stream]
    //   COLUMN:    meta = uint2[K]  {offset/16 of the column block in the stream, entries}
    //   LANE_TILE: meta = uint32[K*S + 1]  offset/16 of sub-block (j, s); sub-blocks are contiguous
    std::vector<uint8_t> image;
    size_t meta_bytes = 0;             // stream starts at image[meta_bytes]
    size_t stream_bytes = 0;
    uint32_t max_unit16 = 0;           // largest column block / sub-block in 16-byte units

    // device binding
    uint8_t *d_image = nullptr;
    uint8_t *d_ws = nullptr;
    celty::WorkspaceLayout ws{};
    int32_t grid = 0, variant = 0, groups = 0, depth = 0, cluster = 0;
    int32_t pairs = -1;                       // fused kernel, two warps per team that take turns at its accumulator:
                                              // -1 = library's choice, 0 = never, 1 = always
    int32_t reg_rows = 0;                     // register-accumulation study: local rows per lane summed in registers
    uint32_t spin_limit = 0;                  // bounded waits inside the kernels: 0 = the library's limit
    int32_t last_grid = 0, last_merge = -1;   // what the tickets in the workspace were last used with
    int32_t mix = -1;       // fused kernel, left-over blocks shared between row parts: 0 never, 1 wherever it is even, -1 where it pays
    int32_t lean = -1;      // fused kernel: 0 = always the build with every option compiled in
    int32_t no_overlap = 0; // fused kernel: 1 = plain launch (no programmatic dependent launch)
    int32_t merge = -1;     // fused kernel: -1 = library's choice, 0 = ordered two-stage sum, 1 = bulk reduce-add
};
