// CUDA half of the library (sm_100a): activation compaction, the two SpMSpV kernels, the decode
// kernels used by parity tests, and the C-ABI entry points that launch them.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <mutex>

#include "celty_internal.h"

using namespace celty;

namespace {

thread_local int g_last_cuda = 0;

#define CELTY_CUDA(expr)                                   \
    do {                                                   \
        cudaError_t err_ = (expr);                         \
        if (err_ != cudaSuccess) {                         \
            g_last_cuda = (int)err_;                       \
            return CELTY_ECUDA;                            \
        }                                                  \
    } while (0)

constexpr unsigned kFull = 0xFFFFFFFFu;
enum : uint32_t { kStatusTimeout = 1u, kStatusBounds = 2u };

struct DeviceInfo { int sms = 0; int max_smem_optin = 0; };

int device_info(DeviceInfo *out)
{
    static std::mutex mu;
    static DeviceInfo cache[64];
    int dev = 0;
    CELTY_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return CELTY_EINVAL;
    std::lock_guard<std::mutex> lock(mu);
    if (cache[dev].sms == 0) {
        CELTY_CUDA(cudaDeviceGetAttribute(&cache[dev].sms, cudaDevAttrMultiProcessorCount, dev));
        CELTY_CUDA(cudaDeviceGetAttribute(&cache[dev].max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    }
    *out = cache[dev];
    return CELTY_OK;
}

// ------------------------------------------------------------------------------------------------
// Run-length decode of one group of 8 entries (Algorithm 1, the per-lane part, done on packed bytes).
// w holds the eight 4-bit runs, entry e in bits 4e..4e+3.  On return byte m of `even` is the
// inclusive sum of runs 0..2m plus the ordinal 2m, byte m of `odd` the same for entry 2m+1, and
// `total` the sum of the 8 runs.  The row of entry e is base + that byte; the largest is 15*8+7 = 127.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void decode_group(uint32_t w, uint32_t &even, uint32_t &odd, uint32_t &total)
{
    const uint32_t lo = w & 0x0F0F0F0Fu;          // runs of entries 0,2,4,6
    const uint32_t hi = (w >> 4) & 0x0F0F0F0Fu;   // runs of entries 1,3,5,7
    const uint32_t p = (lo + hi) * 0x01010101u;   // byte m = runs 0..2m+1 summed
    total = p >> 24;
    odd = p + 0x07050301u;
    even = p - hi + 0x06040200u;
}

__device__ __forceinline__ uint32_t entry_offset(uint32_t even, uint32_t odd, int e)
{
    const uint32_t src = (e & 1) ? odd : even;
    return (src >> (8 * (e >> 1))) & 0xFFu;
}

__device__ __forceinline__ float entry_value(const uint4 &v, int e)
{
    const uint32_t word = e < 2 ? v.x : e < 4 ? v.y : e < 6 ? v.z : v.w;
    const __half2 h2 = *reinterpret_cast<const __half2 *>(&word);
    return (e & 1) ? __high2float(h2) : __low2float(h2);
}

__device__ __forceinline__ uint16_t entry_bits(const uint4 &v, int e)
{
    const uint32_t word = e < 2 ? v.x : e < 4 ? v.y : e < 6 ? v.z : v.w;
    return (uint16_t)((e & 1) ? (word >> 16) : (word & 0xFFFFu));
}

// ------------------------------------------------------------------------------------------------
// Activation compaction (magnitude thresholding, Sections 1 and 2.1): one thread block walks x in
// tiles of 8 values per thread, keeps j iff not(|x_j| <= tau) in FP32, and writes the surviving
// indices and FP16 bit patterns in ascending order.  The same launch clears y when y != nullptr.
// ------------------------------------------------------------------------------------------------
constexpr int kCompactThreads = 1024;

__global__ void __launch_bounds__(kCompactThreads)
k_compact(const uint16_t *__restrict__ x, int K, float tau, int32_t *__restrict__ idx,
          uint16_t *__restrict__ val, int32_t *__restrict__ count, float *__restrict__ y, int M)
{
    __shared__ int warp_tot[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (y) {
        for (int i = tid * 4; i < M; i += kCompactThreads * 4) {
            if (i + 3 < M) {
                *reinterpret_cast<float4 *>(y + i) = make_float4(0.f, 0.f, 0.f, 0.f);
            } else {
                for (int k = i; k < M; ++k) y[k] = 0.f;
            }
        }
    }
    int base = 0;
    for (int tile = 0; tile < K; tile += kCompactThreads * 8) {
        const int e0 = tile + tid * 8;
        uint16_t h[8];
        if (e0 + 8 <= K) {
            const uint4 v = *reinterpret_cast<const uint4 *>(x + e0);
            h[0] = v.x & 0xFFFF; h[1] = v.x >> 16; h[2] = v.y & 0xFFFF; h[3] = v.y >> 16;
            h[4] = v.z & 0xFFFF; h[5] = v.z >> 16; h[6] = v.w & 0xFFFF; h[7] = v.w >> 16;
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) h[k] = (e0 + k < K) ? x[e0 + k] : (uint16_t)0;
        }
        unsigned keep = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float f = __half2float(__ushort_as_half(h[k]));
            if (e0 + k < K && !(fabsf(f) <= tau)) keep |= 1u << k;
        }
        const int cnt = __popc(keep);
        int incl = cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int up = __shfl_up_sync(kFull, incl, d);
            if (lane >= d) incl += up;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            const int t = warp_tot[lane];
            int s = t;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int up = __shfl_up_sync(kFull, s, d);
                if (lane >= d) s += up;
            }
            warp_tot[lane] = s;                     // inclusive totals over warps
        }
        __syncthreads();
        int o = base + (warp ? warp_tot[warp - 1] : 0) + incl - cnt;
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (keep & (1u << k)) {
                idx[o] = e0 + k;
                val[o] = h[k];
                ++o;
            }
        base += warp_tot[31];
        __syncthreads();
    }
    if (tid == 0) *count = base;
}

// ------------------------------------------------------------------------------------------------
// COLUMN layout kernel: the formulation of Sections 3.1-3.3 as published.  A thread block owns a
// slice of the surviving-column list and an M-float accumulator in shared memory.  Each warp takes
// whole columns; per chunk of 256 entries every lane loads 8 values (one 128-bit load) and their 8
// runs, the warp reconstructs rows with the intra-warp prefix sum of Algorithm 1 (per-lane sum,
// five shfl_up steps, back-fill), and scatters value * x_j with shared-memory atomic adds.  The
// accumulator is flushed to y once, with global atomic adds (split-K merge, Section 3.1).
// ------------------------------------------------------------------------------------------------
struct ColumnChunk {
    uint4 v;
    uint32_t even, odd;
    uint32_t row0;        // row of this lane's first entry minus its own offset byte
};

__device__ __forceinline__ ColumnChunk load_column_chunk(const uint8_t *col, uint32_t groups, uint32_t c,
                                                          int lane, uint32_t &carry)
{
    ColumnChunk ch;
    const uint32_t gc = min((uint32_t)kChunkGroups, groups - c * kChunkGroups);
    const uint8_t *chunk = col + (size_t)c * (kChunkGroups * 20);
    uint32_t w = 0;
    ch.v = make_uint4(0, 0, 0, 0);
    if ((uint32_t)lane < gc) {
        ch.v = *reinterpret_cast<const uint4 *>(chunk + 16 * lane);
        w = *reinterpret_cast<const uint32_t *>(chunk + 16 * gc + 4 * lane);
    }
    uint32_t total;
    decode_group(w, ch.even, ch.odd, total);
    // Algorithm 1: inclusive scan over lanes of the rows each lane spans (its runs + its 8 entries)
    const uint32_t span = ((uint32_t)lane < gc) ? total + kGroup : 0u;
    uint32_t sum = span;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t prev = __shfl_up_sync(kFull, sum, d);
        if (lane >= d) sum += prev;
    }
    ch.row0 = carry + sum - span;
    carry += __shfl_sync(kFull, sum, 31);
    return ch;
}

__global__ void __launch_bounds__(256)
k_spmspv_column(const uint2 *__restrict__ meta, const uint8_t *__restrict__ stream,
                const int32_t *__restrict__ idx, const uint16_t *__restrict__ val,
                const int32_t *__restrict__ count, float *__restrict__ y, int M, uint32_t *status)
{
    extern __shared__ float acc[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    for (int i = tid; i < M; i += blockDim.x) acc[i] = 0.f;
    __syncthreads();
    const int n = *count;
    const int p0 = (int)((int64_t)blockIdx.x * n / gridDim.x);
    const int p1 = (int)((int64_t)(blockIdx.x + 1) * n / gridDim.x);
    for (int p = p0 + warp; p < p1; p += nwarps) {
        const int j = idx[p];
        const float xj = __half2float(__ushort_as_half(val[p]));
        const uint2 mj = meta[j];
        const uint8_t *col = stream + (size_t)mj.x * 16;
        const uint32_t nent = mj.y, groups = (nent + kGroup - 1) / kGroup;
        uint32_t carry = 0;
        for (uint32_t c = 0; c * kChunkGroups < groups; ++c) {
            const ColumnChunk ch = load_column_chunk(col, groups, c, lane, carry);
            const uint32_t e0 = (c * kChunkGroups + lane) * kGroup;
#pragma unroll
            for (int e = 0; e < kGroup; ++e) {
                if (e0 + e < nent) {
                    const uint32_t row = ch.row0 + entry_offset(ch.even, ch.odd, e);
                    if (row < (uint32_t)M) atomicAdd(&acc[row], entry_value(ch.v, e) * xj);
                    else atomicOr(status, kStatusBounds);
                }
            }
        }
    }
    __syncthreads();
    for (int i = tid; i < M; i += blockDim.x) {
        const float v = acc[i];
        if (v != 0.f) atomicAdd(&y[i], v);
    }
}

__global__ void k_decode_column(const uint2 *__restrict__ meta, const uint8_t *__restrict__ stream, int j,
                                int32_t *rows, uint16_t *vals, int cap, int32_t *count)
{
    const int lane = threadIdx.x;
    const uint2 mj = meta[j];
    const uint8_t *col = stream + (size_t)mj.x * 16;
    const uint32_t nent = mj.y, groups = (nent + kGroup - 1) / kGroup;
    uint32_t carry = 0;
    for (uint32_t c = 0; c * kChunkGroups < groups; ++c) {
        const ColumnChunk ch = load_column_chunk(col, groups, c, lane, carry);
        const uint32_t e0 = (c * kChunkGroups + lane) * kGroup;
        for (int e = 0; e < kGroup; ++e)
            if (e0 + e < nent && e0 + e < (uint32_t)cap) {
                rows[e0 + e] = (int32_t)(ch.row0 + entry_offset(ch.even, ch.odd, e));
                vals[e0 + e] = entry_bits(ch.v, e);
            }
    }
    if (lane == 0) *count = (int32_t)min(nent, (uint32_t)cap);
}

// ------------------------------------------------------------------------------------------------
// LANE_TILE layout kernel.  Rows are partitioned into tiles of R rows each (the row map tile_row deals
// them out lane by lane and slab by slab) and the rule of Section 3.2 restarts in every tile.  Warp s of a warp group owns slab s (tiles 32s .. 32s+31), lane L owns tile
// 32s+L: each lane walks its own run stream with a running row sum (no cross-lane scan is needed),
// and local row i of lane L lives at accumulator word (s*(R+8) + i)*32 + L, i.e. in bank L -- every
// scatter instruction touches 32 distinct banks, and no two threads ever touch the same word, so the
// accumulation is a plain load / fmaf / store.  The 8 spare rows per slab absorb the zero-valued slots
// that fill a lane's last 16-byte group.  G warp groups per block work on different columns with an
// accumulator each; the flush adds them and merges into y with global atomic adds.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
k_spmspv_lane(const uint32_t *__restrict__ meta, const uint8_t *__restrict__ stream,
              const int32_t *__restrict__ idx, const uint16_t *__restrict__ val,
              const int32_t *__restrict__ count, float *__restrict__ y, int M, int R, int S, int C, int G)
{
    extern __shared__ float acc[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const int slab_words = (R + kTileSlack) * 32, group_words = S * slab_words;
    for (int i = tid; i < G * group_words; i += blockDim.x) acc[i] = 0.f;
    __syncthreads();
    const int g = warp / S, s = warp - g * S;
    const int n = *count;
    const int64_t units = (int64_t)gridDim.x * G, u = (int64_t)blockIdx.x * G + g;
    const int p0 = (int)(u * n / units), p1 = (int)((u + 1) * n / units);
    float *a = acc + g * group_words + s * slab_words + lane;
    for (int p = p0; p < p1; ++p) {
        const int j = idx[p];
        const float xj = __half2float(__ushort_as_half(val[p]));
        const uint8_t *sub = stream + (size_t)meta[(size_t)j * S + s] * 16;
        const uint32_t gl = sub[lane];
        const uint32_t steps = __reduce_max_sync(kFull, gl);
        const uint32_t Gs = __reduce_add_sync(kFull, gl);
        const uint8_t *vbase = sub + kSubHeader, *rbase = vbase + 16 * (size_t)Gs;
        uint32_t slot0 = 0, row = 0;
        for (uint32_t q = 0; q < steps; ++q) {
            const bool active = gl > q;
            const uint32_t ballot = __ballot_sync(kFull, active);
            if (active) {
                const uint32_t slot = slot0 + __popc(ballot & ((1u << lane) - 1u));
                const uint4 v = *reinterpret_cast<const uint4 *>(vbase + 16 * (size_t)slot);
                const uint32_t w = *reinterpret_cast<const uint32_t *>(rbase + 4 * (size_t)slot);
                uint32_t even, odd, total;
                decode_group(w, even, odd, total);
#pragma unroll
                for (int e = 0; e < kGroup; ++e) {
                    float *cell = a + (row + entry_offset(even, odd, e)) * 32;
                    *cell = fmaf(entry_value(v, e), xj, *cell);
                }
                row += total + kGroup;
            }
            slot0 += __popc(ballot);
        }
    }
    __syncthreads();
    for (int w = warp; w < S * R; w += nwarps) {
        const int sl = w / R, i = w - sl * R;
        const int64_t r = tile_row(S, C, sl, lane, i);
        if (r < M) {
            float v = 0.f;
            for (int gg = 0; gg < G; ++gg) v += acc[gg * group_words + sl * slab_words + i * 32 + lane];
            if (v != 0.f) atomicAdd(&y[r], v);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Small batches (N = 2 .. 8 activation vectors against the same matrix).  Section 2.2-2.3 place the method
// against SpMM kernels that need N >= 8 to pay off; here the batch-1 scheme is kept and widened: a column
// is fetched once if ANY of the N activations in it survives the threshold (the union of the surviving
// columns), and every stored entry is multiplied into N accumulators, one per vector, with the activations
// that did not survive replaced by zero (adding value * 0 changes nothing).
//   k_compact_batch  one thread block: union list, and per listed column its N FP16 activations (zero where
//                    dropped), vector-major: val[n * K + position]; clears y.
//   k_spmspv_lane_batch<NB>  lane-tile kernel with plain loads; a block works on one slab of rows (so the
//                    N accumulators of a slab fit shared memory whatever M is), its warps on different columns.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kCompactThreads)
k_compact_batch(const uint16_t *__restrict__ x, int64_t ldx, int N, int K, float tau, int32_t *__restrict__ idx,
                uint16_t *__restrict__ val, int32_t *__restrict__ count, float *__restrict__ y, int64_t ldy, int M)
{
    __shared__ int warp_tot[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int n = 0; n < N; ++n)
        for (int i = tid; i < M; i += kCompactThreads) y[(size_t)n * ldy + i] = 0.f;
    int base = 0;
    for (int tile = 0; tile < K; tile += kCompactThreads) {
        const int j = tile + tid;
        uint16_t h[8];
        bool any = false;
#pragma unroll
        for (int n = 0; n < 8; ++n) {
            h[n] = 0;
            if (n < N && j < K) {
                const uint16_t b = x[(size_t)n * ldx + j];
                if (!(fabsf(__half2float(__ushort_as_half(b))) <= tau)) {
                    h[n] = b;
                    any = true;
                }
            }
        }
        const unsigned bal = __ballot_sync(kFull, any);
        if (lane == 0) warp_tot[warp] = __popc(bal);
        __syncthreads();
        if (warp == 0) {
            const int t = warp_tot[lane];
            int s = t;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int up = __shfl_up_sync(kFull, s, d);
                if (lane >= d) s += up;
            }
            warp_tot[lane] = s;                     // inclusive totals over warps
        }
        __syncthreads();
        if (any) {
            const int o = base + (warp ? warp_tot[warp - 1] : 0) + __popc(bal & ((1u << lane) - 1u));
            idx[o] = j;
#pragma unroll
            for (int n = 0; n < 8; ++n)
                if (n < N) val[(size_t)n * K + o] = h[n];
        }
        base += warp_tot[31];
        __syncthreads();
    }
    if (tid == 0) *count = base;
}

template <int NB>
__global__ void __launch_bounds__(1024)
k_spmspv_lane_batch(const uint32_t *__restrict__ meta, const uint8_t *__restrict__ stream,
                    const int32_t *__restrict__ idx, const uint16_t *__restrict__ val,
                    const int32_t *__restrict__ count, float *__restrict__ y, int64_t ldy, int N, int M, int K, int R,
                    int S, int C)
{
    extern __shared__ float acc[];                  // [warps][NB][(R + 8) * 32]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const int slab_words = (R + kTileSlack) * 32;
    for (int i = tid; i < nwarps * NB * slab_words; i += blockDim.x) acc[i] = 0.f;
    __syncthreads();
    const int s = blockIdx.x % S, kslice = blockIdx.x / S, nK = gridDim.x / S;      // grid = S * nK
    const int n = *count;
    const int64_t units = (int64_t)nK * nwarps, u = (int64_t)kslice * nwarps + warp;
    const int p0 = (int)(u * n / units), p1 = (int)((u + 1) * n / units);
    float *a = acc + (size_t)warp * NB * slab_words + lane;
    for (int p = p0; p < p1; ++p) {
        const int j = idx[p];
        float xv[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) xv[b] = b < N ? __half2float(__ushort_as_half(val[(size_t)b * K + p])) : 0.f;
        const uint8_t *sub = stream + (size_t)meta[(size_t)j * S + s] * 16;
        const uint32_t gl = sub[lane];
        const uint32_t steps = __reduce_max_sync(kFull, gl);
        const uint32_t Gs = __reduce_add_sync(kFull, gl);
        const uint8_t *vbase = sub + kSubHeader, *rbase = vbase + 16 * (size_t)Gs;
        uint32_t slot0 = 0, row = 0;
        for (uint32_t q = 0; q < steps; ++q) {
            const bool active = gl > q;
            const uint32_t ballot = __ballot_sync(kFull, active);
            if (active) {
                const uint32_t slot = slot0 + __popc(ballot & ((1u << lane) - 1u));
                const uint4 v = *reinterpret_cast<const uint4 *>(vbase + 16 * (size_t)slot);
                const uint32_t w = *reinterpret_cast<const uint32_t *>(rbase + 4 * (size_t)slot);
                uint32_t even, odd, total;
                decode_group(w, even, odd, total);
#pragma unroll
                for (int e = 0; e < kGroup; ++e) {
                    const float wv = entry_value(v, e);
                    float *cell = a + (row + entry_offset(even, odd, e)) * 32;
#pragma unroll
                    for (int b = 0; b < NB; ++b) cell[(size_t)b * slab_words] = fmaf(wv, xv[b], cell[(size_t)b * slab_words]);
                }
                row += total + kGroup;
            }
            slot0 += __popc(ballot);
        }
    }
    __syncthreads();
    // merge: the block's warps are added, then one atomic add per (vector, row)
    for (int w = warp; w < R; w += nwarps) {
        const int64_t r = tile_row(S, C, s, lane, w);
        if (r >= M) continue;
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            if (b >= N) break;
            float v = 0.f;
            for (int g = 0; g < nwarps; ++g) v += acc[((size_t)g * NB + b) * slab_words + w * 32 + lane];
            if (v != 0.f) atomicAdd(&y[(size_t)b * ldy + r], v);
        }
    }
}

// scratch[0 .. T] = the column's logical block pointers (entries before each tile), relative to scratch[0]
__global__ void k_decode_lane(const uint32_t *__restrict__ meta, const uint8_t *__restrict__ stream, int j,
                              int S, int C, const uint32_t *__restrict__ scratch, int32_t *rows,
                              uint16_t *vals, int cap, int32_t *count)
{
    const int lane = threadIdx.x & 31, s = threadIdx.x >> 5;
    const uint8_t *sub = stream + (size_t)meta[(size_t)j * S + s] * 16;
    const uint32_t gl = sub[lane];
    const uint32_t steps = __reduce_max_sync(kFull, gl);
    const uint32_t Gs = __reduce_add_sync(kFull, gl);
    const uint8_t *vbase = sub + kSubHeader, *rbase = vbase + 16 * (size_t)Gs;
    const int t = 32 * s + lane, T = 32 * S;
    const uint32_t out0 = scratch[t] - scratch[0];
    const uint32_t nt = scratch[t + 1] - scratch[t];
    uint32_t slot0 = 0, row = 0;
    for (uint32_t q = 0; q < steps; ++q) {
        const bool active = gl > q;
        const uint32_t ballot = __ballot_sync(kFull, active);
        if (active) {
            const uint32_t slot = slot0 + __popc(ballot & ((1u << lane) - 1u));
            const uint4 v = *reinterpret_cast<const uint4 *>(vbase + 16 * (size_t)slot);
            const uint32_t w = *reinterpret_cast<const uint32_t *>(rbase + 4 * (size_t)slot);
            uint32_t even, odd, total;
            decode_group(w, even, odd, total);
            for (int e = 0; e < kGroup; ++e) {
                const uint32_t k = q * kGroup + e;
                if (k < nt && out0 + k < (uint32_t)cap) {
                    rows[out0 + k] = (int32_t)tile_row(S, C, s, lane, row + entry_offset(even, odd, e));
                    vals[out0 + k] = entry_bits(v, e);
                }
            }
            row += total + kGroup;
        }
        slot0 += __popc(ballot);
    }
    if (threadIdx.x == 0) *count = (int32_t)min(scratch[T] - scratch[0], (uint32_t)cap);
}

// Raise a kernel's dynamic shared-memory limit once per device (and again only if a larger size is
// asked for), so that steady-state calls make no attribute calls.  The attribute belongs to the kernel,
// so every entry point that launches a kernel shares that kernel's cache (g_granted_*): two caches for
// one kernel could disagree about what the runtime currently allows.
int g_granted_fused[64], g_granted_lean[2][64], g_granted_fused_extras[64], g_granted_lean_extras[2][64], g_granted_column[64], g_granted_lane[64], g_granted_reg[4][64];

template <typename Kernel>
int ensure_smem(Kernel kernel, size_t bytes, int *granted /* [64], per device */)
{
    int dev = 0;
    CELTY_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return CELTY_EINVAL;
    if ((size_t)granted[dev] >= bytes && granted[dev] > 0) return CELTY_OK;
    CELTY_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
    granted[dev] = (int)bytes;
    return CELTY_OK;
}

#include "celty_fused.cuh"

int launch_compact(const void *x, int64_t K, float tau, int32_t *idx, uint16_t *val, int32_t *count, float *y,
                   int64_t M, cudaStream_t st)
{
    k_compact<<<1, kCompactThreads, 0, st>>>(static_cast<const uint16_t *>(x), (int)K, tau, idx, val, count, y, (int)M);
    CELTY_CUDA(cudaGetLastError());
    return CELTY_OK;
}

// Shape of the fused launch: P row parts of Sc slabs, G teams per slab (teams = G * Sc warps, one accumulator
// slab and one ring of D slots each), clusters of cl thread blocks that add their accumulators on chip.
int plan_fused(const celty_matrix *m, const DeviceInfo &di, FusedPlan *out)
{
    FusedPlan pl{};
    pl.P = m->P;
    pl.Sc = m->Sc;
    if (pl.Sc > 16) return CELTY_EINVAL;      // one warp per team, 16 warps per block
    pl.slot_bytes = (int)round_up((size_t)m->max_unit16 * 16, 128);
    pl.cap = 64;
    const int reg_rows = m->reg_rows;          // register-accumulation study: 256 threads, eight teams at most
    const size_t budget = (size_t)di.max_smem_optin;
    int blocks = std::min(di.sms, kMaxBlocks);  // every block must be resident: they wait for one another's tickets
    if (m->grid > 0) blocks = std::min(blocks, (int)m->grid);
    pl.grid = std::max(blocks, pl.P);           // any number of blocks >= P: parts may differ by one column slice
    if (pl.grid > di.sms) return CELTY_EINVAL;
    // Teams first (each needs its own accumulator), then as many ring slots as still fit (at least two, to
    // keep a copy in flight).  With warp pairs (two warps take turns at a team's accumulator, each with ring slots
    // of its own) there are eight teams at most and an even number of slots.
    auto fit = [&](int pairs) {
        pl.pp = pairs;
        // no more teams than a block can have columns (a tiny layer then leaves half the shared memory free, and
        // the next call's block can set itself up beside this one: 5.25 -> 4.95 us at 1024 x 1024)
        const int64_t cols_per_block = (m->K + std::max(1, pl.grid / pl.P) - 1) / std::max(1, pl.grid / pl.P);
        // Eight teams saturate the shared-memory data path; more of them only pay where a team has a long list of
        // columns to stream (5120 x 13824: 11 teams 4 % faster than 8), and otherwise cost what the block has to
        // add up at the end (4096 x 4096 at 64 rows per tile: 9.1 us with 13 teams, 8.3-8.5 with 7 to 10; 11008 x 4096
        // at 88 rows per tile, 110 columns to a block: 12.7 us with 10 teams, 12.3 with 8 pairs).
        const int most = (reg_rows > 0 || pairs || cols_per_block < 128) ? 8 : 16;
        const int g_cap = (int)std::max<int64_t>(1, std::min<int64_t>(most / pl.Sc, cols_per_block));
        const int g_max = std::max(1, std::min(g_cap, m->groups > 0 ? m->groups : g_cap));
        // two ring slots per team unless asked otherwise: deeper rings measured no faster anywhere, and slower where
        // they only add set-up (4096 x 4096 at 64 rows per tile, eight teams: 8.5 us with two slots, 8.7 with four)
        int d_min = m->depth > 0 ? m->depth : 2, d_max = m->depth > 0 ? m->depth : 2;
        if (pairs) {
            d_min = std::max(2, d_min + (d_min & 1));
            d_max = std::max(d_min, d_max & ~1);
        }
        pl.G = 0;
        for (int g = g_max; g >= 1 && pl.G == 0; --g)
            for (int d = d_max; d >= d_min; --d)
                if ((!pairs || (d & 1) == 0) &&
                    fused_smem_bytes(m->R, (int)m->K, g, pl.Sc, d, pl.slot_bytes, pl.cap) <= budget) {
                    pl.G = g;
                    pl.D = d;
                    break;
                }
    };
    fit(0);
    // Pairs pay where a team has many columns to stream (the hand-over hides the latencies at the head of every
    // sub-block) and cost a little where it has few: measured +7-8 % at 28672 x 8192 and 8192 x 28672, +2 % at
    // 11008 x 4096 and 13824 x 5120, -1 % at 5120 x 5120, -5 % at 4096 x 4096; and they must not cost teams (5120 x 13824
    // runs 11 teams of one warp faster than 8 pairs).  The number of survivors is not known here, so the rule goes
    // by the columns: a dozen or more per team, and no more than eight teams to begin with.
    if (reg_rows == 0 && m->pairs != 0 && pl.G > 0 && pl.Sc <= 8) {             // a pair is warps t and t + 8
        const int teams_per_part = std::max(1, pl.grid / pl.P) * pl.G;
        if (m->pairs > 0 || (pl.G * pl.Sc <= 8 && m->K / teams_per_part >= 12)) {
            const FusedPlan keep = pl;
            fit(1);
            if (pl.G == 0) pl = keep;
        }
    }
    if (pl.G == 0 && m->depth == 0 && fused_smem_bytes(m->R, (int)m->K, 1, pl.Sc, 1, pl.slot_bytes, pl.cap) <= budget) {
        pl.G = 1;
        pl.D = 1;
        pl.pp = 0;
    }
    if (pl.G == 0) return CELTY_EINVAL;
    pl.threads = reg_rows > 0 ? 256 : 512;
    pl.smem = fused_smem_bytes(m->R, (int)m->K, pl.G, pl.Sc, pl.D, pl.slot_bytes, pl.cap);
    pl.merge = (m->merge >= 0 ? m->merge : 1);
    // Clusters (bulk reduce-add merge only, on request): as long as the grid is made of whole clusters, every row
    // part gets at least one, and the device can hold them all at once.
    pl.cl = pl.merge == 1 ? (m->cluster > 0 ? m->cluster : 1) : 1;
    while (pl.cl > 1 && (pl.grid % pl.cl != 0 || pl.grid / pl.cl < pl.P)) pl.cl >>= 1;
    *out = pl;
    return CELTY_OK;
}

// How many clusters of `cl` blocks of the fused kernel (with `smem` bytes of dynamic shared memory each) the
// current device holds at once; asked of the runtime once per (device, cluster size, shared-memory KB).
int max_active_clusters(int cl, size_t smem, int threads, int *out)
{
    struct Entry { int dev, cl, kb, n; };
    static std::mutex mu;
    static Entry cache[64];
    static int used = 0;
    int dev = 0;
    CELTY_CUDA(cudaGetDevice(&dev));
    const int kb = (int)((smem + 1023) / 1024);
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < used; ++i)
        if (cache[i].dev == dev && cache[i].cl == cl && cache[i].kb == kb) {
            *out = cache[i].n;
            return CELTY_OK;
        }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)cl);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = (size_t)kb * 1024;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cl;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    CELTY_CUDA(cudaOccupancyMaxActiveClusters(&n, k_spmspv_fused<false, 0>, &cfg));
    if (used < 64) cache[used++] = Entry{dev, cl, kb, n};
    *out = n;
    return CELTY_OK;
}

// fall back to smaller clusters while the device cannot hold the whole grid of them at once
int fit_clusters_only(FusedPlan *plan)
{
    while (plan->cl > 1) {
        int fit = 0;
        const int rc = max_active_clusters(plan->cl, plan->smem, plan->threads, &fit);
        if (rc) return rc;
        if (fit * plan->cl >= plan->grid) break;
        plan->cl >>= 1;
        while (plan->cl > 1 && (plan->grid % plan->cl != 0 || plan->grid / plan->cl < plan->P)) plan->cl >>= 1;
    }
    return CELTY_OK;
}

// the cluster size the device can hold; then, without clusters, whether the blocks that are left over when the grid
// is dealt to the row parts serve several parts each (FusedParams::mix): only where they can be shared evenly
int fit_clusters(const celty_matrix *m, FusedPlan *plan)
{
    const int rc = fit_clusters_only(plan);
    plan->mix = 1;
    const int left = plan->grid % plan->P;
    if (rc == CELTY_OK && plan->cl == 1 && plan->merge == 1 && m->mix != 0 && left > 0 && plan->P % left == 0) {
        const int mix = plan->P / left;
        // Sharing evens the parts out by 1 / (mix * blocks per part) of the streaming time, and a shared block adds
        // mix times the bytes into y at the end, which takes it mix times as long (the adders in L2 are shared by
        // all blocks): measured 2.2 % faster at 1 / 36 (28672 x 8192), 3 % slower at 1 / 147 (three parts)
        const bool pays = m->mix > 0 || (int64_t)mix * (plan->grid / plan->P) <= 48;
        if (pays && plan->G % mix == 0 && plan->Sc * mix <= 16) plan->mix = mix;
    }
    return rc;
}

}  // namespace

extern "C" int celty_last_cuda_error(void) { return g_last_cuda; }

extern "C" int celty_launch_plan(const celty_matrix *m, int32_t *out, int32_t n)
{
    if (!m || !out || n < 10) return CELTY_EINVAL;
    if (m->layout != CELTY_LAYOUT_LANE_TILE) return CELTY_EINVAL;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    FusedPlan plan;
    rc = plan_fused(m, di, &plan);
    if (rc) return rc;
    rc = ensure_smem(k_spmspv_fused<false, 0>, plan.smem, g_granted_fused);
    if (rc) return rc;
    rc = fit_clusters(m, &plan);
    if (rc) return rc;
    const int32_t v[10] = {plan.grid, plan.threads, (int32_t)plan.smem, plan.G, plan.D, plan.cl, plan.P, plan.Sc,
                           plan.slot_bytes, plan.merge + 16 * plan.pp + 256 * plan.mix};
    for (int i = 0; i < 10; ++i) out[i] = v[i];
    return CELTY_OK;
}


extern "C" int celty_bind_device(celty_matrix *m, void *image_dev, size_t image_bytes, void *workspace_dev,
                                 size_t workspace_bytes, celty_stream_t stream)
{
    if (!m || !image_dev || !workspace_dev) return CELTY_EINVAL;
    if (image_bytes < m->image.size() || workspace_bytes < m->ws.total) return CELTY_ENOMEM;
    if (((uintptr_t)image_dev | (uintptr_t)workspace_dev) & (kAlign - 1)) return CELTY_ENOMEM;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CELTY_CUDA(cudaMemcpyAsync(image_dev, m->image.data(), m->image.size(), cudaMemcpyHostToDevice, st));
    CELTY_CUDA(cudaMemsetAsync(workspace_dev, 0, m->ws.total, st));
    m->d_image = static_cast<uint8_t *>(image_dev);
    m->d_ws = static_cast<uint8_t *>(workspace_dev);
    return CELTY_OK;
}

extern "C" int celty_compact(const void *x_dev, int64_t K, float tau, int32_t *idx_dev, uint16_t *val_dev,
                             int32_t *count_dev, celty_stream_t stream)
{
    if (!x_dev || !idx_dev || !val_dev || !count_dev || K <= 0 || K >= ((int64_t)1 << 31)) return CELTY_EINVAL;
    if (!(tau >= 0.f) || !std::isfinite(tau)) return CELTY_EINVAL;
    if ((uintptr_t)x_dev & 15) return CELTY_EINVAL;
    return launch_compact(x_dev, K, tau, idx_dev, val_dev, count_dev, nullptr, 0, static_cast<cudaStream_t>(stream));
}

namespace {

struct ListInput { const int32_t *idx; const uint16_t *val; const int32_t *count; };
struct SwigluInput { const float *gate_up; uint16_t *h_out; };

int check_epilogue(const celty_matrix *m, const celty_epilogue *ep)
{
    if (!ep || ep->kind == CELTY_EPILOGUE_NONE) return CELTY_OK;
    if (ep->kind == CELTY_EPILOGUE_FP16) return ep->out_fp16 ? CELTY_OK : CELTY_EINVAL;
    if (ep->kind != CELTY_EPILOGUE_SWIGLU) return CELTY_EINVAL;
    if (!ep->out_fp16 || !ep->list_idx || !ep->list_val || !ep->list_count || (m->M & 1)) return CELTY_EINVAL;
    if (!(ep->tau >= 0.f) || !std::isfinite(ep->tau)) return CELTY_EINVAL;
    return CELTY_OK;
}

// The product for every entry point: x thresholded by the kernel (list == nullptr) or the survivors given as a
// list; optional work on y after the merge.
int run_product(celty_matrix *m, const void *x_dev, float tau, const ListInput *list, void *y_dev,
                const celty_epilogue *ep, celty_stream_t stream, const SwigluInput *sw = nullptr)
{
    if (!m || !y_dev || (!x_dev && !list && !sw)) return CELTY_EINVAL;
    if (sw && (!sw->gate_up || ((uintptr_t)sw->gate_up & 15))) return CELTY_EINVAL;
    if (list && (!list->idx || !list->val || !list->count)) return CELTY_EINVAL;
    if (!list && (!(tau >= 0.f) || !std::isfinite(tau))) return CELTY_EINVAL;
    if (((uintptr_t)x_dev | (uintptr_t)y_dev) & 15) return CELTY_EINVAL;
    if (!m->d_image || !m->d_ws) return CELTY_ESTATE;
    int rc = check_epilogue(m, ep);
    if (rc) return rc;
    const bool extras = list || sw || (ep && ep->kind != CELTY_EPILOGUE_NONE);
    // lists and work after the merge exist in the single-launch kernel with the bulk reduce-add merge only
    if (extras && !(m->layout == CELTY_LAYOUT_LANE_TILE && m->variant == 0 && m->merge != 0)) return CELTY_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DeviceInfo di;
    rc = device_info(&di);
    if (rc) return rc;
    uint32_t *status = reinterpret_cast<uint32_t *>(m->d_ws + m->ws.status_off);
    int32_t *count = reinterpret_cast<int32_t *>(status + 1);
    int32_t *idx = reinterpret_cast<int32_t *>(m->d_ws + m->ws.idx_off);
    uint16_t *val = reinterpret_cast<uint16_t *>(m->d_ws + m->ws.val_off);
    float *y = static_cast<float *>(y_dev);
    const uint8_t *stream_base = m->d_image + m->meta_bytes;
    if (m->layout == CELTY_LAYOUT_LANE_TILE && m->variant == 0) {
        FusedPlan plan;
        rc = plan_fused(m, di, &plan);
        if (rc) return rc;
        if (extras && m->reg_rows) return CELTY_EINVAL;
        rc = extras ? ensure_smem(k_spmspv_fused<true, 0>, plan.smem, g_granted_fused_extras)
             : m->reg_rows == 32 ? ensure_smem(k_spmspv_fused<false, 32>, plan.smem, g_granted_reg[0])
             : m->reg_rows == 64 ? ensure_smem(k_spmspv_fused<false, 64>, plan.smem, g_granted_reg[1])
             : m->reg_rows == 96 ? ensure_smem(k_spmspv_fused<false, 96>, plan.smem, g_granted_reg[2])
             : m->reg_rows == 128 ? ensure_smem(k_spmspv_fused<false, 128>, plan.smem, g_granted_reg[3])
                                  : ensure_smem(k_spmspv_fused<false, 0>, plan.smem, g_granted_fused);
        if (rc) return rc;
        rc = fit_clusters(m, &plan);
        if (rc) return rc;
        // the library's default launch has builds of its own (k_spmspv_fused, kLean)
        const int lean = (m->reg_rows == 0 && plan.merge == 1 && plan.cl == 1 && m->lean != 0) ? 1 + plan.pp : 0;
        if (lean) {
            rc = extras ? (lean == 2 ? ensure_smem(k_spmspv_fused<true, 0, 2>, plan.smem, g_granted_lean_extras[1])
                                     : ensure_smem(k_spmspv_fused<true, 0, 1>, plan.smem, g_granted_lean_extras[0]))
                        : (lean == 2 ? ensure_smem(k_spmspv_fused<false, 0, 2>, plan.smem, g_granted_lean[1])
                                     : ensure_smem(k_spmspv_fused<false, 0, 1>, plan.smem, g_granted_lean[0]));
            if (rc) return rc;
        }
        FusedParams fp{};
        if (list) {
            fp.list_idx = list->idx;
            fp.list_val = list->val;
            fp.list_count = list->count;
        }
        if (sw) {
            fp.swiglu_in = sw->gate_up;
            fp.h_out = sw->h_out;
        }
        if (ep && ep->kind != CELTY_EPILOGUE_NONE) {
            fp.ep_kind = ep->kind;
            fp.ep_out = static_cast<uint16_t *>(ep->out_fp16);
            fp.ep_tau = ep->tau;
            fp.ep_idx = ep->list_idx;
            fp.ep_val = ep->list_val;
            fp.ep_count = ep->list_count;
        }
        fp.meta = reinterpret_cast<const uint32_t *>(m->d_image);
        fp.stream = stream_base;
        fp.x = static_cast<const uint16_t *>(x_dev);           // not looked at when the survivors come as a list
        fp.tau = tau;
        fp.y = y;
        fp.idx = idx; fp.val = val; fp.count = count; fp.status = status; fp.tickets = status + 2;
        fp.partials = reinterpret_cast<float *>(m->d_ws + m->ws.partial_off);
        fp.M = (int)m->M; fp.K = (int)m->K; fp.R = m->R; fp.S = (int)m->S; fp.C = m->C;
        fp.G = plan.G; fp.Sc = plan.Sc; fp.P = plan.P; fp.D = plan.D; fp.cl = plan.cl; fp.pp = plan.pp;
        fp.mix = plan.mix;
        fp.slot_bytes = plan.slot_bytes; fp.cap = plan.cap;
        {
            // offset window: as many columns as 32 KB (or the accumulator area, or the table) hold
            const size_t acc_bytes = (size_t)plan.G * plan.Sc * (m->R + kTileSlack) * 128;
            const size_t words = std::min<size_t>(std::min<size_t>(acc_bytes, 32768) / 4, (size_t)m->K * m->S + 4);
            fp.win_cols = (int)std::min<int64_t>(m->K, words >= 8 ? (int64_t)((words - 8) / m->S) : 0);
        }
        fp.merge = plan.merge;
        fp.lay = fused_smem_layout(m->R, (int)m->K, plan.G * plan.Sc, plan.D, plan.slot_bytes, plan.cap);
        fp.clear_rows = (int)(m->M / plan.grid);
        fp.clear_extra = (int)(m->M % plan.grid);
        fp.spin_limit = m->spin_limit ? m->spin_limit : kSpinLimit;
        auto inverse = [](uint64_t units) { return units == 1 ? 0xFFFFFFFFu : (uint32_t)(0x100000000ull / units); };
        const int nclusters = plan.grid / plan.cl;
        fp.units_inv = plan.mix >= 2 ? inverse((uint64_t)(plan.grid / plan.P) * plan.G + plan.G / plan.mix)
                                     : inverse((uint64_t)plan.cl * std::max(1, nclusters / plan.P) * plan.G);
        fp.units_inv_long = inverse((uint64_t)plan.cl * (nclusters / plan.P + 1) * plan.G);
        // the tickets count blocks of one launch shape: start them over when the shape changes
        if (m->last_grid != plan.grid || m->last_merge != plan.merge) {
            CELTY_CUDA(cudaMemsetAsync(m->d_ws + m->ws.status_off + 8, 0, 8, st));
            m->last_grid = plan.grid;
            m->last_merge = plan.merge;
        }
        // Programmatic dependent launch: the kernel may be scheduled while the previous kernel of the stream
        // drains; it waits for that kernel (griddepcontrol.wait) before it reads or writes anything of the call.
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)plan.grid);
        cfg.blockDim = dim3((unsigned)plan.threads);
        cfg.dynamicSmemBytes = plan.smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        int na = 0;
        if (!m->no_overlap) {
            attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[na].val.programmaticStreamSerializationAllowed = 1;
            ++na;
        }
        if (plan.cl > 1) {
            attr[na].id = cudaLaunchAttributeClusterDimension;
            attr[na].val.clusterDim.x = (unsigned)plan.cl;
            attr[na].val.clusterDim.y = 1;
            attr[na].val.clusterDim.z = 1;
            ++na;
        }
        cfg.attrs = attr;
        cfg.numAttrs = na;
        if (extras && lean == 2) CELTY_CUDA(cudaLaunchKernelEx(&cfg, k_spmspv_fused<true, 0, 2>, fp));
        else if (extras && lean == 1) CELTY_CUDA(cudaLaunchKernelEx(&cfg, k_spmspv_fused<true, 0, 1>, fp));
        else if (extras) CELTY_CUDA(cudaLaunchKernelEx(&cfg, k_spmspv_fused<true, 0>, fp));
        else if (m->reg_rows == 32) CELTY_CUDA(cudaLaunchKernelEx(&cfg, k_spmspv_fused<false, 32>, fp));
        else if (m->reg_rows == 64) CELTY_CUDA(cudaLaunchKernelEx(&cfg, k_spmspv_fused<false, 64>, fp));
        else if (m->reg_rows == 96) CELTY_CUDA(cudaLaunchKernelEx(&cfg, k_spmspv_fused<false, 96>, fp));
        else if (m->reg_rows == 128) CELTY_CUDA(cudaLaunchKernelEx(&cfg, k_spmspv_fused<false, 128>, fp));
        else if (lean == 2) CELTY_CUDA(cudaLaunchKernelEx(&cfg, k_spmspv_fused<false, 0, 2>, fp));
        else if (lean == 1) CELTY_CUDA(cudaLaunchKernelEx(&cfg, k_spmspv_fused<false, 0, 1>, fp));
        else CELTY_CUDA(cudaLaunchKernelEx(&cfg, k_spmspv_fused<false, 0>, fp));
        return CELTY_OK;
    }
    // two launches: compaction (which also clears y), then the product.  Sizes are checked and the
    // shared-memory limit is raised before the first launch, so that an error return leaves y untouched.
    if (m->layout == CELTY_LAYOUT_COLUMN) {
        const size_t smem = (size_t)m->M * 4;
        if (smem > (size_t)di.max_smem_optin) return CELTY_EINVAL;
        rc = ensure_smem(k_spmspv_column, smem, g_granted_column);
        if (rc) return rc;
        rc = launch_compact(x_dev, m->K, tau, idx, val, count, y, m->M, st);
        if (rc) return rc;
        const int per_sm = (int)std::max<size_t>(1, std::min<size_t>(8, (size_t)(di.max_smem_optin) / (smem + 1024)));
        const int grid = m->grid > 0 ? m->grid : di.sms * per_sm;
        k_spmspv_column<<<grid, 256, smem, st>>>(reinterpret_cast<const uint2 *>(m->d_image), stream_base, idx, val,
                                                  count, y, (int)m->M, status);
    } else {
        const size_t group_bytes = (size_t)m->S * (m->R + kTileSlack) * 32 * 4;
        if (group_bytes > (size_t)di.max_smem_optin) return CELTY_EINVAL;
        int G = (int)std::min<size_t>((size_t)di.max_smem_optin / group_bytes, (size_t)(32 / m->S));
        G = std::max(1, std::min(G, m->groups > 0 ? m->groups : (int)std::max<int64_t>(1, 8 / m->S)));
        const size_t smem = group_bytes * G;
        rc = ensure_smem(k_spmspv_lane, smem, g_granted_lane);
        if (rc) return rc;
        rc = launch_compact(x_dev, m->K, tau, idx, val, count, y, m->M, st);
        if (rc) return rc;
        const int grid = m->grid > 0 ? m->grid : di.sms;
        k_spmspv_lane<<<grid, 32 * (int)m->S * G, smem, st>>>(reinterpret_cast<const uint32_t *>(m->d_image),
                                                              stream_base, idx, val, count, y, (int)m->M, m->R,
                                                              (int)m->S, m->C, G);
    }
    CELTY_CUDA(cudaGetLastError());
    return CELTY_OK;
}

}  // namespace

extern "C" int celty_spmspv(celty_matrix *m, const void *x_dev, float tau, void *y_dev, celty_stream_t stream)
{
    if (!x_dev) return CELTY_EINVAL;
    return run_product(m, x_dev, tau, nullptr, y_dev, nullptr, stream);
}

extern "C" int celty_spmspv_ex(celty_matrix *m, const void *x_dev, float tau, void *y_dev, const celty_epilogue *ep,
                               celty_stream_t stream)
{
    if (!x_dev) return CELTY_EINVAL;
    return run_product(m, x_dev, tau, nullptr, y_dev, ep, stream);
}

extern "C" int celty_spmspv_swiglu(celty_matrix *m, const float *gate_up_dev, float tau, void *y_dev, void *h_out_dev,
                                   const celty_epilogue *ep, celty_stream_t stream)
{
    const SwigluInput sw{gate_up_dev, static_cast<uint16_t *>(h_out_dev)};
    return run_product(m, nullptr, tau, nullptr, y_dev, ep, stream, &sw);
}

extern "C" int celty_spmspv_list(celty_matrix *m, const int32_t *idx_dev, const uint16_t *val_dev,
                                 const int32_t *count_dev, void *y_dev, const celty_epilogue *ep, celty_stream_t stream)
{
    const ListInput list{idx_dev, val_dev, count_dev};
    return run_product(m, nullptr, 0.f, &list, y_dev, ep, stream);
}

// ------------------------------------------------------------------------------------------------
// celty_spmspv_static: scratch in a file-scope device array instead of a caller-provided workspace,
// for callers that cannot allocate device memory.  Layout of the array: [256 B header: status, count]
// [int32 idx[kStaticMaxK]][uint16 val[kStaticMaxK]].
// ------------------------------------------------------------------------------------------------
namespace {

constexpr int64_t kStaticMaxK = 32768;
constexpr size_t kStaticScratchBytes = 256 + (size_t)kStaticMaxK * 4 + (size_t)kStaticMaxK * 2;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code the array's name is only a stand-in: the device address comes from the runtime, once
// per device, with that device current.
int static_scratch_address(uint8_t **out)
{
    static std::mutex mu;
    static uint8_t *address[64];
    int dev = 0;
    CELTY_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return CELTY_EINVAL;
    std::lock_guard<std::mutex> lock(mu);
    if (!address[dev]) {
        void *p = nullptr;
        CELTY_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
        address[dev] = static_cast<uint8_t *>(p);
    }
    *out = address[dev];
    return CELTY_OK;
}

}  // namespace

extern "C" int celty_spmspv_static(const celty_matrix *m, const void *image_dev, const void *x_dev, float tau,
                                   void *y_dev, celty_stream_t stream)
{
    if (!m || !image_dev || !x_dev || !y_dev) return CELTY_EINVAL;
    if (!(tau >= 0.f) || !std::isfinite(tau)) return CELTY_EINVAL;
    if (((uintptr_t)x_dev | (uintptr_t)y_dev | (uintptr_t)image_dev) & 15) return CELTY_EINVAL;
    if (m->layout != CELTY_LAYOUT_LANE_TILE) return CELTY_EINVAL;
    if (m->K > kStaticMaxK) return CELTY_ELIMIT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    uint8_t *scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc) return rc;
    // every check comes before the first launch: an error return leaves y untouched
    const size_t group_bytes = (size_t)m->S * (m->R + kTileSlack) * 32 * 4;
    if (group_bytes > (size_t)di.max_smem_optin || m->S > 32) return CELTY_ELIMIT;
    const int G = (int)std::max<size_t>(1, std::min<size_t>((size_t)di.max_smem_optin / group_bytes,
                                                             (size_t)std::max<int64_t>(1, 8 / m->S)));
    const size_t smem = group_bytes * G;
    rc = ensure_smem(k_spmspv_lane, smem, g_granted_lane);
    if (rc) return rc;
    int32_t *count = reinterpret_cast<int32_t *>(scratch) + 1;
    int32_t *idx = reinterpret_cast<int32_t *>(scratch + 256);
    uint16_t *val = reinterpret_cast<uint16_t *>(scratch + 256 + (size_t)kStaticMaxK * 4);
    float *y = static_cast<float *>(y_dev);
    rc = launch_compact(x_dev, m->K, tau, idx, val, count, y, m->M, st);     // also clears y
    if (rc) return rc;
    const uint8_t *image = static_cast<const uint8_t *>(image_dev);
    k_spmspv_lane<<<di.sms, 32 * (int)m->S * G, smem, st>>>(reinterpret_cast<const uint32_t *>(image),
                                                            image + m->meta_bytes, idx, val, count, y, (int)m->M, m->R,
                                                            (int)m->S, m->C, G);
    CELTY_CUDA(cudaGetLastError());
    return CELTY_OK;
}

extern "C" int celty_spmspv_batch(celty_matrix *m, const void *x_dev, int64_t ldx, int32_t N, float tau, void *y_dev,
                                  int64_t ldy, void *list_scratch_dev, size_t scratch_bytes, celty_stream_t stream)
{
    if (!m || !x_dev || !y_dev || !list_scratch_dev) return CELTY_EINVAL;
    if (N < 1 || N > 8 || ldx < m->K || ldy < m->M) return CELTY_EINVAL;
    if (!(tau >= 0.f) || !std::isfinite(tau)) return CELTY_EINVAL;
    if (m->layout != CELTY_LAYOUT_LANE_TILE) return CELTY_EINVAL;
    if (!m->d_image) return CELTY_ESTATE;
    // scratch: count (256 bytes), int32 idx[K], FP16 val[8][K]
    const size_t need = 256 + round_up((size_t)m->K * 4, 256) + (size_t)8 * m->K * 2;
    if (scratch_bytes < need || ((uintptr_t)list_scratch_dev & 255)) return CELTY_ENOMEM;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Measured, the widened kernels below lose to the single-vector kernel called N times at every N (N accumulators
    // per warp leave room for fewer warps, and the union of N activation patterns is nearly every column from N = 4
    // on): unless the two-launch variant is asked for, the batch is N launches of the single-launch kernel, where the
    // handle has its workspace and every row of x and y starts on a 16-byte boundary.
    if (m->variant == 0 && m->d_ws && !(((uintptr_t)x_dev | (uintptr_t)(ldx * 2) | (uintptr_t)y_dev | (uintptr_t)(ldy * 4)) & 15)) {
        for (int32_t n = 0; n < N; ++n) {
            const int rc1 = celty_spmspv(m, static_cast<const uint16_t *>(x_dev) + (size_t)n * ldx, tau,
                                         static_cast<float *>(y_dev) + (size_t)n * ldy, stream);
            if (rc1) return rc1;
        }
        return CELTY_OK;
    }
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    uint8_t *sc = static_cast<uint8_t *>(list_scratch_dev);
    int32_t *count = reinterpret_cast<int32_t *>(sc);
    int32_t *idx = reinterpret_cast<int32_t *>(sc + 256);
    uint16_t *val = reinterpret_cast<uint16_t *>(sc + 256 + round_up((size_t)m->K * 4, 256));
    const int NB = N <= 2 ? 2 : N <= 4 ? 4 : 8;
    const size_t slab_bytes = (size_t)(m->R + kTileSlack) * 32 * 4;
    const int warps = (int)std::min<size_t>(16, (size_t)di.max_smem_optin / (slab_bytes * NB));
    if (warps < 1) return CELTY_ELIMIT;
    const size_t smem = slab_bytes * NB * warps;
    static int granted[3][64];
    auto launch = [&](auto kernel, int slot) -> int {
        const int r = ensure_smem(kernel, smem, granted[slot]);
        if (r) return r;
        k_compact_batch<<<1, kCompactThreads, 0, st>>>(static_cast<const uint16_t *>(x_dev), ldx, N, (int)m->K, tau, idx, val,
                                                       count, static_cast<float *>(y_dev), ldy, (int)m->M);
        const int nK = std::max(1, di.sms / (int)m->S);
        kernel<<<(int)m->S * nK, 32 * warps, smem, st>>>(reinterpret_cast<const uint32_t *>(m->d_image),
                                                          m->d_image + m->meta_bytes, idx, val, count,
                                                          static_cast<float *>(y_dev), ldy, N, (int)m->M, (int)m->K, m->R,
                                                          (int)m->S, m->C);
        return CELTY_OK;
    };
    rc = NB == 2 ? launch(k_spmspv_lane_batch<2>, 0) : NB == 4 ? launch(k_spmspv_lane_batch<4>, 1)
                                                             : launch(k_spmspv_lane_batch<8>, 2);
    if (rc) return rc;
    CELTY_CUDA(cudaGetLastError());
    return CELTY_OK;
}

extern "C" int celty_spmspv_host(celty_matrix *m, const void *x_host, float tau, void *y_host, void *x_stage_dev,
                                 void *y_stage_dev, celty_stream_t stream)
{
    if (!m || !x_host || !y_host || !x_stage_dev || !y_stage_dev) return CELTY_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CELTY_CUDA(cudaMemcpyAsync(x_stage_dev, x_host, (size_t)m->K * 2, cudaMemcpyHostToDevice, st));
    const int rc = celty_spmspv(m, x_stage_dev, tau, y_stage_dev, stream);
    if (rc) return rc;
    CELTY_CUDA(cudaMemcpyAsync(y_host, y_stage_dev, (size_t)m->M * 4, cudaMemcpyDeviceToHost, st));
    CELTY_CUDA(cudaStreamSynchronize(st));
    return CELTY_OK;
}

extern "C" int celty_last_compaction(const celty_matrix *m, const int32_t **count_dev, const int32_t **idx_dev,
                                     const uint16_t **val_dev)
{
    if (!m) return CELTY_EINVAL;
    if (!m->d_ws) return CELTY_ESTATE;
    if (count_dev) *count_dev = reinterpret_cast<const int32_t *>(m->d_ws + m->ws.status_off) + 1;
    if (idx_dev) *idx_dev = reinterpret_cast<const int32_t *>(m->d_ws + m->ws.idx_off);
    if (val_dev) *val_dev = reinterpret_cast<const uint16_t *>(m->d_ws + m->ws.val_off);
    return CELTY_OK;
}

extern "C" int celty_decode_device(celty_matrix *m, int64_t col, int32_t *rows_dev, uint16_t *vals_dev, int64_t cap,
                                   int32_t *count_dev, celty_stream_t stream)
{
    if (!m || !rows_dev || !vals_dev || !count_dev || col < 0 || col >= m->K || cap < 0 || cap > 0x7FFFFFFF)
        return CELTY_EINVAL;
    if (!m->d_image || !m->d_ws) return CELTY_ESTATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint8_t *stream_base = m->d_image + m->meta_bytes;
    if (m->layout == CELTY_LAYOUT_COLUMN) {
        k_decode_column<<<1, 32, 0, st>>>(reinterpret_cast<const uint2 *>(m->d_image), stream_base, (int)col, rows_dev,
                                          vals_dev, (int)cap, count_dev);
    } else {
        uint32_t *scratch = reinterpret_cast<uint32_t *>(m->d_ws + m->ws.scratch_off);
        CELTY_CUDA(cudaMemcpyAsync(scratch, &m->block_ptr[(size_t)col * m->T], (size_t)(m->T + 1) * 4,
                                   cudaMemcpyHostToDevice, st));
        k_decode_lane<<<1, 32 * (int)m->S, 0, st>>>(reinterpret_cast<const uint32_t *>(m->d_image), stream_base,
                                                    (int)col, (int)m->S, m->C, scratch, rows_dev, vals_dev,
                                                    (int)cap, count_dev);
    }
    CELTY_CUDA(cudaGetLastError());
    return CELTY_OK;
}

extern "C" int celty_last_status(celty_matrix *m, celty_stream_t stream)
{
    if (!m) return CELTY_EINVAL;
    if (!m->d_ws) return CELTY_ESTATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t word = 0;
    CELTY_CUDA(cudaMemcpyAsync(&word, m->d_ws + m->ws.status_off, 4, cudaMemcpyDeviceToHost, st));
    CELTY_CUDA(cudaStreamSynchronize(st));
    if (word) {
        // also reset the fused kernel's tickets, which a run that gave up may have left mid-count
        CELTY_CUDA(cudaMemsetAsync(m->d_ws + m->ws.status_off, 0, 4, st));
        CELTY_CUDA(cudaMemsetAsync(m->d_ws + m->ws.status_off + 8, 0, 8, st));
        CELTY_CUDA(cudaStreamSynchronize(st));
        m->last_grid = 0;
    }
    if (word & kStatusTimeout) return CELTY_ETIMEOUT;
    if (word & kStatusBounds) return CELTY_EBOUNDS;
    return CELTY_OK;
}
