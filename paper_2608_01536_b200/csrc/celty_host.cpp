// Host half of the library: offline packing into RLC-CSC (Section 3.2, Fig. 2(a)), the handle,
// host-side decoding for round-trip tests and byte accounting.  No CUDA calls in this file.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <memory>
#include <new>

#include "celty_internal.h"

using namespace celty;

namespace {

inline bool kept(const uint16_t *W, int64_t ldw, const uint8_t *mask, int64_t K, int64_t r, int64_t j)
{
    return mask ? mask[r * K + j] != 0 : (W[r * ldw + j] & 0x7FFFu) != 0;
}

// Pack the 4-bit runs of 8 consecutive entries, entry e in bits 4e .. 4e+3.
inline uint32_t pack_runs(const uint8_t *r, int n)
{
    uint32_t w = 0;
    for (int e = 0; e < n; ++e) w |= (uint32_t)(r[e] & 15u) << (4 * e);
    return w;
}

struct Logical {                 // one run per byte, block-major (column, tile), rows ascending
    std::vector<uint16_t> vals;
    std::vector<uint8_t> runs;
};

// Slabs S, local rows per tile R and chunk C of the LANE_TILE row map for M rows (tile_rows = 0: library's
// choice).  Up to 128 local rows per lane: a lane's run stream is then ~8 groups per column at 50% density,
// and eight or nine teams with their accumulators and rings fit one SM's shared memory.  Measured on B200 over
// the configured shapes, S = ceil(M / 4096) was the best or within 6% of the best slab count everywhere.
// On very tall layers (6 slabs or more) the streaming loop dominates, and what counts there is that eight warp
// teams fit one SM's 227 KB of shared memory (accumulator slab + two ring slots each): when the density of the
// kept weights makes the sub-blocks too large for that at 128 local rows, fewer rows per tile (in steps of 8, down
// to 96) and correspondingly more slabs are taken: 104 rows at 70% of the weights kept, 120 at 50%, 128 at 30% on
// 28672 x 8192 (measured: 44.4 us against 53.0 at 128 rows and 47.0 at 96; 37.1 against 37.7; no change).
void choose_shape(int64_t M, int64_t K, double density, int tile_rows, int64_t *S_out, int32_t *R_out, int32_t *C_out)
{
    const int64_t Q = (M + 31) / 32;                                  // groups of 32 rows
    int64_t S, R;
    if (tile_rows > 0) {
        R = tile_rows;
        S = (Q + R - 1) / R;
    } else {
        S = std::max<int64_t>(1, (M + 4095) / 4096);
        // A layer of one slab and few columns streams for so short a time that the merge dominates: two slabs
        // halve what every block adds up and adds into y (and the contributors per row), for twice as many
        // sub-blocks of half the size.  Measured at 4096 x 4096: 8.3 us against 8.8; at 4096 x 11008, where a team
        // has five sub-blocks to stream, no gain, so the rule stops short of it.
        if (S == 1 && Q >= 32 && K <= 6144) S = 2;
        auto rows_for = [&](int64_t slabs) { return std::max<int64_t>(16, ((Q + slabs - 1) / slabs + 15) / 16 * 16); };
        auto teams_that_fit = [&](int64_t rows) {
            const double entries = 32.0 * rows * density;             // of one sub-block, mean; + 3.5 sigma for the largest
            const double largest = entries + 3.5 * std::sqrt(entries * (1.0 - density)) + 32 * 3.5;  // + group filling
            const double slot = std::ceil((kSubHeader + 2.5 * largest) / 128.0) * 128.0;
            const double misc = 2.0 * ((K + 31) / 32) * 4 + 17.0 * ((K + 255) / 256) * 4 + 1024;
            return (int64_t)((232448.0 - misc) / ((rows + kTileSlack) * 128.0 + 2.0 * slot + 1024.0));
        };
        R = rows_for(S);
        if (S >= 6)
            for (int fewer = 1; fewer <= 4 && teams_that_fit(R) < 8 && R > 32; ++fewer) {
                R -= 8;                                                // in steps of 8 rows: the chunk of the row map halves
                S = (Q + R - 1) / R;
            }
    }
    *S_out = S;
    *R_out = (int32_t)R;
    // chunks of 16 groups = 2 KB of consecutive rows of y: the merge adds them with one bulk copy each, and 2 KB
    // copies measured 3-4% faster per call than 512-byte ones on the mid-size shapes
    *C_out = R % 16 == 0 ? 16 : R % 8 == 0 ? 8 : R % 4 == 0 ? 4 : 1;
}

// Build the COLUMN image: meta uint2[K] {off16, entries}, then per column its chunks of up to 32
// groups; chunk = [groups x 16 B values][groups x 4 B runs]; column block padded to 16 bytes.
void pack_column(celty_matrix *m, const Logical &lg)
{
    const int64_t K = m->K;
    m->meta_bytes = round_up((size_t)K * 8, kAlign);
    std::vector<uint64_t> off(K + 1, 0);
    for (int64_t j = 0; j < K; ++j) {
        uint64_t n = m->block_ptr[j + 1] - m->block_ptr[j];
        uint64_t groups = (n + kGroup - 1) / kGroup;
        off[j + 1] = off[j] + round_up((size_t)groups * 20, 16);
        m->max_unit16 = std::max<uint32_t>(m->max_unit16, (uint32_t)((off[j + 1] - off[j]) / 16));
    }
    m->stream_bytes = round_up((size_t)off[K], kAlign);
    m->image.assign(m->meta_bytes + m->stream_bytes, 0);
    uint32_t *meta = reinterpret_cast<uint32_t *>(m->image.data());
    uint8_t *stream = m->image.data() + m->meta_bytes;
    for (int64_t j = 0; j < K; ++j) {
        const uint64_t e0 = m->block_ptr[j], n = m->block_ptr[j + 1] - e0;
        meta[2 * j] = (uint32_t)(off[j] / 16);
        meta[2 * j + 1] = (uint32_t)n;
        const uint64_t groups = (n + kGroup - 1) / kGroup;
        uint8_t *col = stream + off[j];
        for (uint64_t g = 0; g < groups; ++g) {
            const uint64_t c = g / kChunkGroups, gl = g % kChunkGroups;
            const uint64_t gc = std::min<uint64_t>(kChunkGroups, groups - c * kChunkGroups);
            uint8_t *chunk = col + c * (kChunkGroups * 20);
            const int cnt = (int)std::min<uint64_t>(kGroup, n - g * kGroup);
            std::memcpy(chunk + 16 * gl, &lg.vals[e0 + g * kGroup], (size_t)cnt * 2);
            uint32_t w = pack_runs(&lg.runs[e0 + g * kGroup], cnt);
            std::memcpy(chunk + 16 * gc + 4 * gl, &w, 4);
        }
    }
}

// Build the LANE_TILE image: meta uint32[K*S + 1] (offset/16 of each sub-block), then per
// (column j, slab s) a sub-block
//   [48 B header: 32 x u8 groups of lane L's tile 32s+L, u32 vectors | steps << 16][G x 16 B values][G x 4 B runs],
// padded to 16 bytes,
// G = sum of the lanes' group counts.  Vectors are stored step-major: for step q = 0, 1, ... the
// lanes that still have a q-th group, in lane order, so that a warp reads one contiguous span per step.
void pack_lane_tile(celty_matrix *m, const Logical &lg)
{
    const int64_t K = m->K, S = m->S, T = m->T;
    m->meta_bytes = round_up((size_t)(K * S + 1) * 4, kAlign);
    std::vector<uint64_t> off((size_t)(K * S + 1), 0);
    for (int64_t j = 0; j < K; ++j)
        for (int64_t s = 0; s < S; ++s) {
            uint64_t G = 0;
            for (int L = 0; L < 32; ++L) {
                int64_t t = 32 * s + L;
                if (t >= T) break;
                uint64_t n = m->block_ptr[j * T + t + 1] - m->block_ptr[j * T + t];
                G += (n + kGroup - 1) / kGroup;
            }
            size_t b = j * S + s;
            off[b + 1] = off[b] + round_up(kSubHeader + (size_t)G * 20, 16);
            m->max_unit16 = std::max<uint32_t>(m->max_unit16, (uint32_t)((off[b + 1] - off[b]) / 16));
        }
    m->stream_bytes = round_up((size_t)off[K * S], kAlign);
    m->image.assign(m->meta_bytes + m->stream_bytes, 0);
    uint32_t *meta = reinterpret_cast<uint32_t *>(m->image.data());
    uint8_t *stream = m->image.data() + m->meta_bytes;
    for (size_t b = 0; b <= (size_t)(K * S); ++b) meta[b] = (uint32_t)(off[b] / 16);
    for (int64_t j = 0; j < K; ++j)
        for (int64_t s = 0; s < S; ++s) {
            uint8_t *sub = stream + off[j * S + s];
            uint64_t e0[32], n[32], g[32], G = 0, steps = 0;
            for (int L = 0; L < 32; ++L) {
                int64_t t = 32 * s + L;
                if (t < T) {
                    e0[L] = m->block_ptr[j * T + t];
                    n[L] = m->block_ptr[j * T + t + 1] - e0[L];
                } else {
                    e0[L] = 0; n[L] = 0;
                }
                g[L] = (n[L] + kGroup - 1) / kGroup;
                sub[L] = (uint8_t)g[L];
                G += g[L];
                steps = std::max(steps, g[L]);
            }
            {
                const uint32_t gs = (uint32_t)G | ((uint32_t)steps << 16);
                std::memcpy(sub + 32, &gs, 4);
            }
            uint8_t *vbase = sub + kSubHeader, *rbase = vbase + 16 * G;
            uint64_t slot = 0;
            for (uint64_t q = 0; q < steps; ++q)
                for (int L = 0; L < 32; ++L) {
                    if (g[L] <= q) continue;
                    const int cnt = (int)std::min<uint64_t>(kGroup, n[L] - q * kGroup);
                    std::memcpy(vbase + 16 * slot, &lg.vals[e0[L] + q * kGroup], (size_t)cnt * 2);
                    uint32_t w = pack_runs(&lg.runs[e0[L] + q * kGroup], cnt);
                    std::memcpy(rbase + 4 * slot, &w, 4);
                    ++slot;
                }
        }
}

}  // namespace

extern "C" int celty_encode(const uint16_t *W, int64_t ldw, const uint8_t *mask, int64_t M, int64_t K,
                            const celty_encode_opts *opts, celty_matrix **out)
{
    if (!W || !out || M <= 0 || K <= 0 || ldw < K || M > kMaxM || K >= ((int64_t)1 << 31)) return CELTY_EINVAL;
    celty_encode_opts o = {4, CELTY_LAYOUT_LANE_TILE, 0, 0};
    if (opts) o = *opts;
    if (o.run_bits != 4 || o.slabs_per_block < 0 || o.slabs_per_block > 15) return CELTY_EINVAL;
    if (o.layout == CELTY_LAYOUT_COLUMN && o.slabs_per_block != 0) return CELTY_EINVAL;
    if (o.layout != CELTY_LAYOUT_COLUMN && o.layout != CELTY_LAYOUT_LANE_TILE) return CELTY_EINVAL;
    if (o.layout == CELTY_LAYOUT_COLUMN && o.tile_rows != 0) return CELTY_EINVAL;
    if (o.layout == CELTY_LAYOUT_LANE_TILE && (o.tile_rows < 0 || o.tile_rows > kMaxTileRows)) return CELTY_EINVAL;
    *out = nullptr;
    try {
        std::unique_ptr<celty_matrix> owner(new celty_matrix());   // released to the caller only on success
        celty_matrix *m = owner.get();
        m->M = M; m->K = K; m->layout = o.layout;
        if (o.layout == CELTY_LAYOUT_COLUMN) {
            m->R = (int32_t)M; m->T = 1; m->S = 1;
        } else {
            double density = 0.5;
            if (o.tile_rows == 0 && M > 5 * 4096) {                   // only very tall layers look at the density
                uint64_t kept_weights = 0;
                for (int64_t r = 0; r < M; ++r)
                    for (int64_t j = 0; j < K; ++j) kept_weights += kept(W, ldw, mask, K, r, j) ? 1 : 0;
                density = (double)kept_weights / ((double)M * (double)K);
            }
            choose_shape(M, K, density, o.tile_rows, &m->S, &m->R, &m->C);
            m->T = 32 * m->S;
            if (m->S > 32) return CELTY_EINVAL;                 // one warp per slab, 32 warps per block
        }
        const int64_t R = m->R, T = m->T;
        const bool lane_tile = m->layout == CELTY_LAYOUT_LANE_TILE;
        // local row i of tile t -> row of W (COLUMN: the one tile is the column itself)
        auto row_of = [&](int64_t t, int64_t i) { return lane_tile ? tile_row(m->S, m->C, t / 32, t % 32, i) : i; };
        // Pass 1: one sweep over the rows of W keeps, per column, the last kept row; the gap before a
        // kept weight is split into floor(gap/16) pads and a run of gap mod 16 (Section 3.2).
        std::vector<uint32_t> cnt((size_t)(K * T), 0);
        std::vector<int32_t> last((size_t)K);
        uint64_t total = 0;
        for (int64_t t = 0; t < T; ++t) {
            std::fill(last.begin(), last.end(), -1);
            for (int64_t i = 0; i < R; ++i) {
                const int64_t r = row_of(t, i);
                if (r >= M) break;                                    // a tile's rows grow with i
                for (int64_t j = 0; j < K; ++j) {
                    if (!kept(W, ldw, mask, K, r, j)) continue;
                    const uint32_t gap = (uint32_t)(i - last[j] - 1);
                    cnt[j * T + t] += (gap >> 4) + 1;
                    total += (gap >> 4) + 1;
                    m->n_pad += gap >> 4;
                    m->nnz += 1;
                    last[j] = (int32_t)i;
                }
            }
        }
        if (total > 0xFFFFFFFFull) return CELTY_EINVAL;
        m->block_ptr.resize((size_t)(K * T + 1));
        uint32_t acc = 0;
        for (int64_t b = 0; b < K * T; ++b) { m->block_ptr[b] = acc; acc += cnt[b]; }
        m->block_ptr[K * T] = acc;
        // Pass 2: same sweep, now writing (value, run) pairs at each block's cursor.
        Logical lg;
        lg.vals.assign((size_t)total + kGroup, 0);
        lg.runs.assign((size_t)total + kGroup, 0);
        m->pad_bits.assign((size_t)(total + 7) / 8, 0);
        std::vector<uint32_t> cur(m->block_ptr.begin(), m->block_ptr.end() - 1);
        for (int64_t t = 0; t < T; ++t) {
            std::fill(last.begin(), last.end(), -1);
            for (int64_t i = 0; i < R; ++i) {
                const int64_t r = row_of(t, i);
                if (r >= M) break;
                for (int64_t j = 0; j < K; ++j) {
                    if (!kept(W, ldw, mask, K, r, j)) continue;
                    uint32_t gap = (uint32_t)(i - last[j] - 1);
                    uint32_t &c = cur[j * T + t];
                    for (; gap > 15; gap -= 16) {
                        lg.vals[c] = 0; lg.runs[c] = 15;
                        m->pad_bits[c >> 3] |= (uint8_t)(1u << (c & 7));
                        ++c;
                    }
                    lg.vals[c] = W[r * ldw + j]; lg.runs[c] = (uint8_t)gap; ++c;
                    last[j] = (int32_t)i;
                }
            }
        }
        if (m->layout == CELTY_LAYOUT_COLUMN) pack_column(m, lg); else pack_lane_tile(m, lg);
        const int64_t spb = o.slabs_per_block > 0 ? o.slabs_per_block : kSlabsPerBlock;
        m->P = (int32_t)((m->S + spb - 1) / spb);
        m->Sc = (int32_t)((m->S + m->P - 1) / m->P);
        m->ws = workspace_layout(K, T, m->layout == CELTY_LAYOUT_LANE_TILE ? (int64_t)m->Sc * m->R * 32 : 0);
        *out = owner.release();
        return CELTY_OK;
    } catch (const std::bad_alloc &) {
        return CELTY_ENOMEM;
    }
}

extern "C" void celty_destroy(celty_matrix *m) { delete m; }

extern "C" int celty_clone(const celty_matrix *m, celty_matrix **out)
{
    if (!m || !out) return CELTY_EINVAL;
    *out = nullptr;
    try {
        std::unique_ptr<celty_matrix> copy(new celty_matrix(*m));
        copy->d_image = nullptr;                  // the copy starts unbound, with the library's launch choices
        copy->d_ws = nullptr;
        copy->last_grid = 0;
        copy->last_merge = -1;
        *out = copy.release();
        return CELTY_OK;
    } catch (const std::bad_alloc &) {
        return CELTY_ENOMEM;
    }
}

extern "C" int celty_info(const celty_matrix *m, int64_t *M, int64_t *K, int64_t *nnz, int64_t *n_pad,
                          int64_t *compressed_bytes, int32_t *layout, int32_t *tile_rows)
{
    if (!m) return CELTY_EINVAL;
    if (M) *M = m->M;
    if (K) *K = m->K;
    if (nnz) *nnz = m->nnz;
    if (n_pad) *n_pad = m->n_pad;
    if (compressed_bytes) *compressed_bytes = (m->nnz + m->n_pad) * 5 / 2 + 4 * (m->K + 1);
    if (layout) *layout = m->layout;
    if (tile_rows) *tile_rows = m->layout == CELTY_LAYOUT_COLUMN ? 0 : m->R;
    return CELTY_OK;
}

extern "C" int celty_row_map(const celty_matrix *m, int32_t *slabs, int32_t *tile_rows, int32_t *chunk)
{
    if (!m) return CELTY_EINVAL;
    if (slabs) *slabs = (int32_t)m->S;
    if (tile_rows) *tile_rows = m->R;
    if (chunk) *chunk = m->C;
    return CELTY_OK;
}

// Decode column `col` from the packed image (not from the encoder's temporaries).
extern "C" int celty_decode_host(const celty_matrix *m, int64_t col, int32_t *rows, uint16_t *vals,
                                 uint8_t *runs, uint8_t *is_pad, int64_t cap, int64_t *n_out)
{
    if (!m || col < 0 || col >= m->K) return CELTY_EINVAL;
    const int64_t T = m->T;
    const int64_t n = (int64_t)m->block_ptr[(col + 1) * T] - (int64_t)m->block_ptr[col * T];
    if (n_out) *n_out = n;
    if (n > cap) return CELTY_ENOMEM;
    const uint8_t *stream = m->image.data() + m->meta_bytes;
    const uint32_t *meta = reinterpret_cast<const uint32_t *>(m->image.data());
    int64_t o = 0;
    // A pad cannot be told from a kept +0 that follows 15 dropped rows by looking at the image, so
    // the flag comes from the bit the encoder recorded for the entry's logical position.
    auto emit = [&](uint64_t logical, int64_t row, uint16_t v, uint8_t run) {
        if (rows) rows[o] = (int32_t)row;
        if (vals) vals[o] = v;
        if (runs) runs[o] = run;
        if (is_pad) is_pad[o] = (m->pad_bits[logical >> 3] >> (logical & 7)) & 1u;
        ++o;
    };
    if (m->layout == CELTY_LAYOUT_COLUMN) {
        const uint8_t *colp = stream + (size_t)meta[2 * col] * 16;
        const int64_t groups = (n + kGroup - 1) / kGroup;
        int64_t s = 0;
        for (int64_t e = 0; e < n; ++e) {
            const int64_t g = e / kGroup, c = g / kChunkGroups, gl = g % kChunkGroups;
            const int64_t gc = std::min<int64_t>(kChunkGroups, groups - c * kChunkGroups);
            const uint8_t *chunk = colp + c * (kChunkGroups * 20);
            uint16_t v; uint32_t w;
            std::memcpy(&v, chunk + 16 * gl + 2 * (e % kGroup), 2);
            std::memcpy(&w, chunk + 16 * gc + 4 * gl, 4);
            const uint8_t run = (w >> (4 * (e % kGroup))) & 15u;
            s += run;
            emit((uint64_t)m->block_ptr[col] + e, s + e, v, run);
        }
    } else {
        for (int64_t sl = 0; sl < m->S; ++sl) {
            const uint8_t *sub = stream + (size_t)meta[col * m->S + sl] * 16;
            int64_t G = 0;
            for (int L = 0; L < 32; ++L) G += sub[L];
            const uint8_t *vbase = sub + kSubHeader, *rbase = vbase + 16 * G;
            for (int L = 0; L < 32; ++L) {
                const int64_t t = 32 * sl + L;
                if (t >= T) break;
                const int64_t nt = (int64_t)m->block_ptr[col * T + t + 1] - (int64_t)m->block_ptr[col * T + t];
                int64_t s = 0;
                for (int64_t e = 0; e < nt; ++e) {
                    const int64_t q = e / kGroup;
                    // slot of (step q, lane L): all lanes' groups of earlier steps + lower lanes of this step
                    int64_t slot = 0;
                    for (int L2 = 0; L2 < 32; ++L2) slot += std::min<int64_t>(sub[L2], q) + (L2 < L && sub[L2] > q ? 1 : 0);
                    uint16_t v; uint32_t w;
                    std::memcpy(&v, vbase + 16 * slot + 2 * (e % kGroup), 2);
                    std::memcpy(&w, rbase + 4 * slot, 4);
                    const uint8_t run = (w >> (4 * (e % kGroup))) & 15u;
                    s += run;
                    emit((uint64_t)m->block_ptr[col * T + t] + e, tile_row(m->S, m->C, sl, L, s + e), v, run);
                }
            }
        }
    }
    return CELTY_OK;
}

extern "C" int celty_host_image(const celty_matrix *m, const void **image, size_t *image_bytes, size_t *stream_offset)
{
    if (!m) return CELTY_EINVAL;
    if (image) *image = m->image.data();
    if (image_bytes) *image_bytes = m->image.size();
    if (stream_offset) *stream_offset = m->meta_bytes;
    return CELTY_OK;
}

extern "C" int celty_device_bytes(const celty_matrix *m, size_t *image_bytes, size_t *workspace_bytes)
{
    if (!m) return CELTY_EINVAL;
    if (image_bytes) *image_bytes = m->image.size();
    if (workspace_bytes) *workspace_bytes = m->ws.total;
    return CELTY_OK;
}

extern "C" int celty_fetched_bytes(const celty_matrix *m, const int32_t *idx, int64_t n, int64_t *stream_bytes,
                                   int64_t *total_bytes)
{
    if (!m || (!idx && n > 0) || n < 0) return CELTY_EINVAL;
    const uint32_t *meta = reinterpret_cast<const uint32_t *>(m->image.data());
    int64_t sb = 0, mb = 0;
    for (int64_t p = 0; p < n; ++p) {
        const int64_t j = idx[p];
        if (j < 0 || j >= m->K) return CELTY_EINVAL;
        if (m->layout == CELTY_LAYOUT_COLUMN) {
            const int64_t groups = ((int64_t)meta[2 * j + 1] + kGroup - 1) / kGroup;
            sb += (int64_t)round_up((size_t)groups * 20, 16);
            mb += 8;
        } else {
            sb += ((int64_t)meta[(j + 1) * m->S] - (int64_t)meta[j * m->S]) * 16;
            mb += 4 * (m->S + 1);
        }
    }
    if (stream_bytes) *stream_bytes = sb;
    // x read once, the list written (4-byte index + 2-byte value), y written once.  Scratch traffic of
    // the split-K merge (per-block partial sums) is not counted: it is overhead, not work.
    if (total_bytes) *total_bytes = sb + mb + 2 * m->K + 6 * n + 4 * m->M;
    return CELTY_OK;
}

extern "C" int celty_stored_entries(const celty_matrix *m, const int32_t *idx, int64_t n, int64_t *entries)
{
    if (!m || (!idx && n > 0) || n < 0 || !entries) return CELTY_EINVAL;
    int64_t e = 0;
    for (int64_t p = 0; p < n; ++p) {
        const int64_t j = idx[p];
        if (j < 0 || j >= m->K) return CELTY_EINVAL;
        e += (int64_t)m->block_ptr[(j + 1) * m->T] - (int64_t)m->block_ptr[j * m->T];
    }
    *entries = e;
    return CELTY_OK;
}

extern "C" int celty_layout_stats(const celty_matrix *m, int64_t *sub_blocks, int64_t *steps, int64_t *groups)
{
    if (!m) return CELTY_EINVAL;
    if (m->layout != CELTY_LAYOUT_LANE_TILE) return CELTY_EINVAL;
    const uint32_t *meta = reinterpret_cast<const uint32_t *>(m->image.data());
    const uint8_t *stream = m->image.data() + m->meta_bytes;
    int64_t nb = 0, st = 0, gr = 0;
    for (int64_t b = 0; b < m->K * m->S; ++b) {
        uint32_t hw;
        std::memcpy(&hw, stream + (size_t)meta[b] * 16 + 32, 4);      // vectors | steps << 16 (see kSubHeader)
        ++nb;
        st += hw >> 16;
        gr += hw & 0xFFFFu;
    }
    if (sub_blocks) *sub_blocks = nb;
    if (steps) *steps = st;
    if (groups) *groups = gr;
    return CELTY_OK;
}

extern "C" int celty_shard_columns(int64_t K, int32_t world, int32_t rank, int64_t *k_begin, int64_t *k_end)
{
    if (K <= 0 || world < 1 || rank < 0 || rank >= world || !k_begin || !k_end) return CELTY_EINVAL;
    // groups of 8 columns (16 bytes of FP16 activations) dealt as evenly as they go: a shard's slice of x then
    // starts on the 16-byte boundary the kernels ask for
    const int64_t groups = (K + 7) / 8, base = groups / world, extra = groups % world;
    const int64_t g0 = rank * base + std::min<int64_t>(rank, extra), g1 = g0 + base + (rank < extra ? 1 : 0);
    *k_begin = std::min<int64_t>(K, g0 * 8);
    *k_end = std::min<int64_t>(K, g1 * 8);
    return CELTY_OK;
}

extern "C" int celty_count_entries(const uint8_t *mask, int64_t ldm, int64_t M, int64_t K, int run_bits,
                                   int64_t *nnz, int64_t *n_pad)
{
    if (!mask || M <= 0 || K <= 0 || ldm < K || run_bits < 1 || run_bits > 8) return CELTY_EINVAL;
    // rows outermost (the mask is row-major); gap[j] = dropped rows of column j since its last kept row
    std::vector<int64_t> gap;
    try {
        gap.assign((size_t)K, 0);
    } catch (const std::bad_alloc &) {
        return CELTY_ENOMEM;
    }
    int64_t kept = 0, pads = 0;
    for (int64_t i = 0; i < M; ++i) {
        const uint8_t *row = mask + i * ldm;
        for (int64_t j = 0; j < K; ++j) {
            if (!row[j]) {
                ++gap[(size_t)j];
                continue;
            }
            ++kept;
            pads += gap[(size_t)j] >> run_bits;      // a padding entry covers 2^run_bits rows: its run and itself
            gap[(size_t)j] = 0;
        }
    }
    if (nnz) *nnz = kept;
    if (n_pad) *n_pad = pads;
    return CELTY_OK;
}

extern "C" int celty_set_launch(celty_matrix *m, int32_t grid, int32_t variant, int32_t groups, int32_t depth,
                                int32_t cluster)
{
    if (!m || grid < 0 || variant < 0 || variant > 509 || groups < 0 || groups > 16 || depth < 0 || depth > 16 ||
        !(cluster == 0 || cluster == 1 || cluster == 2 || cluster == 4))
        return CELTY_EINVAL;
    m->grid = grid;
    // variant: bit 0 selects the two-launch path; 2 / 4 force the ordered two-stage / the bulk reduce-add merge
    m->merge = (variant & 2) ? 0 : (variant & 4) ? 1 : -1;
    m->no_overlap = (variant & 8) ? 1 : 0;
    m->variant = variant & 1;
    m->pairs = (variant & 16) ? 1 : (variant & 32) ? 0 : -1;
    m->mix = (variant & 64) ? 0 : (variant & 128) ? 1 : -1;
    m->lean = (variant & 256) ? 0 : -1;
    m->groups = groups;
    m->depth = depth;
    m->cluster = cluster;
    return CELTY_OK;
}

extern "C" int celty_set_register_rows(celty_matrix *m, int32_t rows)
{
    if (!m || !(rows == 0 || rows == 32 || rows == 64 || rows == 96 || rows == 128)) return CELTY_EINVAL;
    m->reg_rows = rows;
    return CELTY_OK;
}

extern "C" int celty_set_wait_limit(celty_matrix *m, uint32_t polls)
{
    if (!m) return CELTY_EINVAL;
    m->spin_limit = polls;
    return CELTY_OK;
}

extern "C" const char *celty_strerror(int status)
{
    switch (status) {
        case CELTY_OK: return "ok";
        case CELTY_EINVAL: return "invalid argument";
        case CELTY_ENOMEM: return "out of memory or buffer too small";
        case CELTY_ECUDA: return "CUDA runtime error";
        case CELTY_ESTATE: return "handle is not bound to device memory";
        case CELTY_ETIMEOUT: return "a bounded wait inside a kernel ran out";
        case CELTY_EBOUNDS: return "a decoded index was out of range";
        case CELTY_ELIMIT: return "size exceeds the fixed scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}
