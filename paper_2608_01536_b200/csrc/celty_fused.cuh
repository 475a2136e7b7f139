// The single-launch SpMSpV kernel for the LANE_TILE layout (included by celty_kernels.cu inside its
// anonymous namespace, after decode_group / entry_value).
//
// One launch does the whole call (Sections 3.1-3.3):
//   a0  every block clears its share of y and takes an "arrived" ticket;
//   a1  every block thresholds all of x (K <= a few 10k values, served by L2), ranks the survivors with
//       a block scan and keeps the ranks that belong to it -- the list is balanced over blocks by count;
//       the block that owns a rank also writes it to the global list (index, value, count) for the API;
//   a2  each warp streams the sub-blocks (column j, slab s) of its columns from HBM into its own ring of
//       shared-memory slots with bulk asynchronous copies (cp.async.bulk + mbarrier complete_tx), D deep;
//   a3  each lane decodes its own tile's runs on packed bytes and keeps a running row;
//   a4  value * x_j is accumulated with fmaf into the lane's private bank of the warp's accumulator;
//   a5  after the "arrived" tickets show that all of y is cleared, the block adds its G accumulators and
//       merges them into y with 128-bit vector reductions; the last block to leave resets the tickets.
//
// Rows are split over P parts (blockIdx % P) of Sc slabs each, columns over gridDim/P slices; inside a
// block G warp groups take different columns.  All waits are bounded: when one runs out the kernel sets
// kStatusTimeout in the status word and carries on to a clean exit.

struct FusedParams {
    const uint32_t *meta;      // [K*S + 1] offset/16 of sub-block (j, s) in the stream
    const uint8_t *stream;
    const uint16_t *x;         // K FP16
    float tau;
    float *y;                  // M
    int32_t *idx;              // global compacted list (API output)
    uint16_t *val;
    int32_t *count;
    uint32_t *status;
    uint32_t *tickets;         // [0] arrived (y cleared), [1] departed
    int M, K, R, S, T;
    int G, Sc, P, D;
    int slot_bytes;            // ring slot size, multiple of 128
    int cap;                   // items per warp group per round
};

constexpr uint32_t kSpinLimit = 1u << 21;

// Phase timestamps for development builds (-DCELTY_TRACE): thread 0 of every block stores clock64()
// at phase k into trace[blockIdx.x * 16 + k].  Compiled out of the product.
#ifdef CELTY_TRACE
__device__ long long *g_celty_trace = nullptr;
#define CELTY_MARK(k)                                                        \
    do {                                                                     \
        if (threadIdx.x == 0 && g_celty_trace) g_celty_trace[blockIdx.x * 16 + (k)] = clock64(); \
    } while (0)
#else
#define CELTY_MARK(k)
#endif

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Wait for a phase of an mbarrier with an iteration limit; false = gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > 256) __nanosleep(128);
    }
    return false;
}

// Bulk asynchronous copy global -> shared (1-D, no tensor map, no multicast); src, dst and bytes are
// multiples of 16.  Completion is signalled on the mbarrier as transferred bytes.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void red_add_v4(float *p, float a, float b, float c, float d)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// 8 run-length decoded accumulations of one lane: cells are word (row)*32 of the lane's bank.
// All loads are issued before the stores: the 8 rows of a group are distinct, so this is the same
// result as 8 dependent read-modify-writes but leaves the memory pipeline full.
__device__ __forceinline__ void accumulate_group(uint32_t cell_base, const uint4 &v, uint32_t even, uint32_t odd,
                                                 float xj)
{
    // cell address = cell_base + 128 * offset byte: one dot-product-accumulate per entry
    uint32_t a[8];
    a[0] = __dp4a(even, 0x00000080u, cell_base);
    a[1] = __dp4a(odd, 0x00000080u, cell_base);
    a[2] = __dp4a(even, 0x00008000u, cell_base);
    a[3] = __dp4a(odd, 0x00008000u, cell_base);
    a[4] = __dp4a(even, 0x00800000u, cell_base);
    a[5] = __dp4a(odd, 0x00800000u, cell_base);
    a[6] = __dp4a(even, 0x80000000u, cell_base);
    a[7] = __dp4a(odd, 0x80000000u, cell_base);
    float c[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) asm volatile("ld.shared.f32 %0, [%1];" : "=f"(c[e]) : "r"(a[e]));
    const __half2 h01 = *reinterpret_cast<const __half2 *>(&v.x), h23 = *reinterpret_cast<const __half2 *>(&v.y);
    const __half2 h45 = *reinterpret_cast<const __half2 *>(&v.z), h67 = *reinterpret_cast<const __half2 *>(&v.w);
    const float2 f01 = __half22float2(h01), f23 = __half22float2(h23), f45 = __half22float2(h45),
                 f67 = __half22float2(h67);
    c[0] = fmaf(f01.x, xj, c[0]); c[1] = fmaf(f01.y, xj, c[1]);
    c[2] = fmaf(f23.x, xj, c[2]); c[3] = fmaf(f23.y, xj, c[3]);
    c[4] = fmaf(f45.x, xj, c[4]); c[5] = fmaf(f45.y, xj, c[5]);
    c[6] = fmaf(f67.x, xj, c[6]); c[7] = fmaf(f67.y, xj, c[7]);
#pragma unroll
    for (int e = 0; e < 8; ++e) asm volatile("st.shared.f32 [%0], %1;" ::"r"(a[e]), "f"(c[e]) : "memory");
}

__global__ void __launch_bounds__(1024) k_spmspv_fused(const FusedParams p)
{
    extern __shared__ __align__(128) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthreads = blockDim.x, nwarps = nthreads >> 5;
    const int slab_words = (p.R + kTileSlack) * 32;
    // ---- shared memory carve-up (offsets mirror fused_smem_bytes on the host)
    float *acc = reinterpret_cast<float *>(smem);
    size_t off = (size_t)nwarps * slab_words * 4;
    uint8_t *ring = smem + off;
    off += (size_t)nwarps * p.D * p.slot_bytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + off);
    off += (size_t)nwarps * p.D * 8;
    int2 *items = reinterpret_cast<int2 *>(smem + off);           // [G][cap] {column, x bits}
    off += (size_t)p.G * p.cap * 8;
    uint2 *imeta = reinterpret_cast<uint2 *>(smem + off);         // [nwarps][cap] {offset/16, bytes}
    off += (size_t)nwarps * p.cap * 8;
    int *misc = reinterpret_cast<int *>(smem + off);              // [0..31] warp totals, [32] n, [40..] group bounds
    off += 512;
    uint8_t *kb = smem + off;                                     // keep bits, one byte per 8 activations

    const int part = blockIdx.x % p.P, kslice = blockIdx.x / p.P, nK = gridDim.x / p.P;
    const int g = warp / p.Sc, sl = warp - g * p.Sc;
    const int s = part * p.Sc + sl;                               // this warp's slab; may be >= S (idle)

    CELTY_MARK(0);
    // ---- a0: clear the accumulators, clear this block's share of y, announce it
    for (int i = tid; i < nwarps * slab_words; i += nthreads) acc[i] = 0.f;
    {
        const int r0 = (int)((int64_t)blockIdx.x * p.M / gridDim.x), r1 = (int)((int64_t)(blockIdx.x + 1) * p.M / gridDim.x);
        for (int i = r0 + tid; i < r1; i += nthreads) p.y[i] = 0.f;
    }
    if (lane == 0) {
        for (int d = 0; d < p.D; ++d) mbar_init(smem_u32(&bars[warp * p.D + d]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) atomicAdd(&p.tickets[0], 1u);
    CELTY_MARK(1);

    // ---- a1: threshold all of x; kb[q] = keep bits of activations 8q .. 8q+7
    const int ngroups = (p.K + 7) >> 3;
    for (int q = tid; q < ngroups; q += nthreads) {
        uint32_t h[4];
        if (8 * q + 8 <= p.K) {
            const uint4 v = *reinterpret_cast<const uint4 *>(p.x + 8 * q);
            h[0] = v.x; h[1] = v.y; h[2] = v.z; h[3] = v.w;
        } else {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t lo = (8 * q + 2 * k < p.K) ? p.x[8 * q + 2 * k] : 0u;
                const uint32_t hi = (8 * q + 2 * k + 1 < p.K) ? p.x[8 * q + 2 * k + 1] : 0u;
                h[k] = lo | (hi << 16);
            }
        }
        uint32_t keep = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint16_t bits = (uint16_t)((k & 1) ? (h[k >> 1] >> 16) : (h[k >> 1] & 0xFFFFu));
            const float f = __half2float(__ushort_as_half(bits));
            if (8 * q + k < p.K && !(fabsf(f) <= p.tau)) keep |= 1u << k;
        }
        kb[q] = (uint8_t)keep;
    }
    __syncthreads();
    CELTY_MARK(2);
    // each thread owns a contiguous run of groups, so ranks follow the column order
    const int per = (ngroups + nthreads - 1) / nthreads;
    const int q0 = min(ngroups, tid * per), q1 = min(ngroups, q0 + per);
    int mine = 0;
    for (int q = q0; q < q1; ++q) mine += __popc((uint32_t)kb[q]);
    int incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int up = __shfl_up_sync(kFull, incl, d);
        if (lane >= d) incl += up;
    }
    if (lane == 31) misc[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int t = lane < nwarps ? misc[lane] : 0;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int up = __shfl_up_sync(kFull, t, d);
            if (lane >= d) t += up;
        }
        misc[lane] = t;                                           // inclusive totals over warps
        if (lane == 31) misc[32] = t;
    }
    __syncthreads();
    const int n = misc[32];
    const int base = (warp ? misc[warp - 1] : 0) + incl - mine;   // rank of this thread's first survivor
    // group gg of this block owns ranks [bound(gg), bound(gg+1)), balanced over all nK * G groups
    const int64_t units = (int64_t)nK * p.G;
    if (tid <= p.G) misc[40 + tid] = (int)(((int64_t)kslice * p.G + tid) * n / units);
    if (blockIdx.x == 0 && tid == 0) *p.count = n;
    __syncthreads();
    CELTY_MARK(3);
    const int r_lo = misc[40], r_hi = misc[40 + p.G];
    int longest = 0;
    for (int gg = 0; gg < p.G; ++gg) longest = max(longest, misc[41 + gg] - misc[40 + gg]);
    const int rounds = (longest + p.cap - 1) / p.cap;

    float *my_acc = acc + (size_t)warp * slab_words;
    const uint32_t cell0 = smem_u32(my_acc) + 4u * lane;
    uint32_t issued = 0, consumed = 0;                            // ring positions of this warp (all rounds)
    bool failed = false;

    for (int round = 0; round < rounds; ++round) {
        // ---- items of this round: rank r of group gg goes to items[gg][r - bound(gg) - round*cap]
        if (base < r_hi && base + mine > r_lo) {
            int r = base;
            for (int q = q0; q < q1; ++q) {
                uint32_t bits = kb[q];
                while (bits) {
                    const int k = __ffs(bits) - 1;
                    bits &= bits - 1;
                    if (r >= r_lo && r < r_hi) {
                        int gg = 0;
                        while (r >= misc[41 + gg]) ++gg;
                        const int local = r - misc[40 + gg] - round * p.cap;
                        const int j = 8 * q + k;
                        if (local >= 0 && local < p.cap) items[gg * p.cap + local] = make_int2(j, (int)p.x[j]);
                        if (round == 0 && part == 0) {
                            p.idx[r] = j;
                            p.val[r] = p.x[j];
                        }
                    }
                    ++r;
                }
            }
        }
        __syncthreads();
        CELTY_MARK(4);
        const int cnt = max(0, min(p.cap, misc[41 + g] - misc[40 + g] - round * p.cap));
        if (s < p.S && !failed) {
            // ---- a2: sub-block addresses of my items, then keep D copies in flight
            for (int i = lane; i < cnt; i += 32) {
                const int j = items[g * p.cap + i].x;
                const uint32_t o0 = p.meta[(size_t)j * p.S + s], o1 = p.meta[(size_t)j * p.S + s + 1];
                imeta[warp * p.cap + i] = make_uint2(o0, (o1 - o0) * 16u);
            }
            __syncwarp();
            auto issue = [&](int i) {
                const uint32_t slot = issued % (uint32_t)p.D;
                const uint2 im = imeta[warp * p.cap + i];
                const uint32_t bar = smem_u32(&bars[warp * p.D + slot]);
                mbar_expect_tx(bar, im.y);
                bulk_load(smem_u32(ring + ((size_t)warp * p.D + slot) * p.slot_bytes), p.stream + (size_t)im.x * 16, im.y,
                          bar);
                ++issued;
            };
            if (lane == 0)
                for (int i = 0; i < min(cnt, p.D); ++i) issue(i);
            issued = __shfl_sync(kFull, issued, 0);
            CELTY_MARK(5);
            for (int i = 0; i < cnt; ++i) {
                const uint32_t slot = consumed % (uint32_t)p.D, parity = (consumed / (uint32_t)p.D) & 1u;
                if (!mbar_wait_bounded(smem_u32(&bars[warp * p.D + slot]), parity)) failed = true;
                failed = __any_sync(kFull, failed);
                if (failed) break;
                if (i == 0) CELTY_MARK(6);
                ++consumed;
                const uint8_t *sub = ring + ((size_t)warp * p.D + slot) * p.slot_bytes;
                const float xj = __half2float(__ushort_as_half((uint16_t)items[g * p.cap + i].y));
                // ---- a3 + a4
                const uint32_t gl = sub[lane];
                const uint32_t steps = __reduce_max_sync(kFull, gl);
                const uint32_t Gs = __reduce_add_sync(kFull, gl);
                const uint8_t *vbase = sub + 32, *rbase = vbase + 16 * Gs;
                uint32_t slot0 = 0, cell = cell0;
                for (uint32_t q = 0; q < steps; ++q) {
                    const bool active = gl > q;
                    const uint32_t ballot = __ballot_sync(kFull, active);
                    if (active) {
                        const uint32_t k = slot0 + __popc(ballot & ((1u << lane) - 1u));
                        const uint4 v = *reinterpret_cast<const uint4 *>(vbase + 16 * k);
                        const uint32_t w = *reinterpret_cast<const uint32_t *>(rbase + 4 * k);
                        uint32_t even, odd, total;
                        decode_group(w, even, odd, total);
                        accumulate_group(cell, v, even, odd, xj);
                        cell += (total + kGroup) * 128u;
                    }
                    slot0 += __popc(ballot);
                }
                __syncwarp();
                if (lane == 0 && i + p.D < cnt) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    issue(i + p.D);
                }
            }
            issued = __shfl_sync(kFull, issued, 0);
        }
        __syncthreads();                                          // items / imeta are rewritten next round
        CELTY_MARK(7);
    }
    if (failed) {
        // give copies that are still in flight a last (bounded) chance to land before the block exits
        for (; consumed < issued; ++consumed)
            mbar_wait_bounded(smem_u32(&bars[warp * p.D + consumed % (uint32_t)p.D]), (consumed / (uint32_t)p.D) & 1u);
        if (lane == 0) atomicOr(p.status, kStatusTimeout);
    }

    // ---- a5: all of y must be cleared before anybody adds to it
    if (tid == 0) {
        bool ok = false;
        for (uint32_t it = 0; it < kSpinLimit; ++it) {
            if (ld_acquire_u32(&p.tickets[0]) >= gridDim.x) { ok = true; break; }
            __nanosleep(64);
        }
        if (!ok) atomicOr(p.status, kStatusTimeout);
    }
    __syncthreads();
    CELTY_MARK(8);
    // lanes keep their bank; warp w walks (slab, 4 consecutive local rows) units
    const int quads = (p.R + 3) / 4;
    for (int u = warp; u < p.Sc * quads; u += nwarps) {
        const int fsl = u / quads, i0 = (u - fsl * quads) * 4;
        const int fs = part * p.Sc + fsl, t = 32 * fs + lane;
        if (fs >= p.S || t >= p.T) continue;
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        for (int gg = 0; gg < p.G; ++gg) {
            const float *a = acc + (size_t)(gg * p.Sc + fsl) * slab_words + lane;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (i0 + k < p.R) v[k] += a[(i0 + k) * 32];
        }
        const int row = t * p.R + i0;
        if ((p.R & 3) == 0 && row + 3 < p.M) {
            if (v[0] != 0.f || v[1] != 0.f || v[2] != 0.f || v[3] != 0.f) red_add_v4(p.y + row, v[0], v[1], v[2], v[3]);
        } else {
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (i0 + k < p.R && row + k < p.M && v[k] != 0.f) atomicAdd(p.y + row + k, v[k]);
        }
    }
    __syncthreads();
    CELTY_MARK(9);
    if (tid == 0) {
        __threadfence();
        const uint32_t t = atomicAdd(&p.tickets[1], 1u);
        if (t == gridDim.x - 1) {                                  // last one out resets both tickets
            atomicExch(&p.tickets[0], 0u);
            atomicExch(&p.tickets[1], 0u);
        }
    }
    CELTY_MARK(10);
}

struct FusedPlan {
    int G, Sc, P, D, slot_bytes, cap, threads, grid;
    size_t smem;
};

inline size_t fused_smem_bytes(int R, int K, int G, int Sc, int D, int slot_bytes, int cap)
{
    const size_t nwarps = (size_t)G * Sc;
    size_t b = nwarps * (size_t)(R + kTileSlack) * 32 * 4;
    b += nwarps * D * (size_t)slot_bytes;
    b += nwarps * D * 8;
    b += (size_t)G * cap * 8;
    b += nwarps * cap * 8;
    b += 512;
    b += round_up((size_t)(K + 7) / 8, 16);
    return b;
}
