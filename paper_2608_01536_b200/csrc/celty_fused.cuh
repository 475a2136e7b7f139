// The single-launch SpMSpV kernel for the LANE_TILE layout (included by celty_kernels.cu inside its
// anonymous namespace, after decode_group).
//
// One launch does the whole call (Sections 3.1-3.3):
//   a1  every block thresholds all of x (K <= a few 10k values, served by L2) into one keep bit per
//       activation; every warp then ranks the survivors by itself (popcounts + one warp scan) and looks
//       up the columns whose ranks belong to it -- the list is balanced over all warp groups by count.
//       The warp that owns a rank also writes it to the global list (index, value, count) for the API;
//   a2  each warp streams the sub-blocks (column j, slab s) of its columns from HBM into its own ring of
//       shared-memory slots with bulk asynchronous copies (cp.async.bulk + mbarrier complete_tx), D deep;
//   a3  each lane decodes its own tile's runs on packed bytes and keeps a running row;
//   a4  value * x_j is accumulated with fmaf into the lane's private bank of the warp's accumulator;
//   a5  the block adds its G accumulators and stores them as one partial vector; after a bounded
//       grid-wide ticket barrier each block sums a share of the rows over all partials in a fixed order
//       and stores y.  No atomics on y, no clearing of y, and the result is deterministic.
//
// Rows are split over P parts (blockIdx % P) of Sc slabs each, columns over gridDim/P slices; inside a
// block G warp groups take different columns.  Every block must be resident at once (grid <= SM count)
// because of the ticket barrier.  All waits are bounded: when one runs out the kernel sets
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
    uint32_t *tickets;         // [0] partial stored, [1] departed
    float *partials;           // gridDim.x vectors of Sc * R * 32 floats (accumulator layout)
    int M, K, R, S, T;
    int G, Sc, P, D;
    long long stream_bytes;    // size of the entry stream (used by the self-checks of development builds)
    int slot_bytes;            // ring slot size, multiple of 128
    int cap;                   // items a warp looks up per batch
    int flags;                 // bit 0: three-stage software pipeline in the step loop
};

constexpr uint32_t kSpinLimit = 1u << 21;

// Development builds only (compiled out of the product):
//   -DCELTY_TRACE  thread 0 of every block stores clock64() at phase k into trace[blockIdx.x * 16 + k];
//   -DCELTY_GUARD  every index is range-checked; a failed check records (value, count) at
//                  trace[192 * 16 + 2 * code] and the access is skipped or redirected, so that a wrong
//                  index shows up as data instead of as a fault.
#if defined(CELTY_TRACE) || defined(CELTY_GUARD)
__constant__ long long *g_celty_trace = nullptr;
#endif
#ifdef CELTY_TRACE
#define CELTY_MARK(k)                                                        \
    do {                                                                     \
        if (threadIdx.x == 0 && g_celty_trace) g_celty_trace[blockIdx.x * 16 + (k)] = clock64(); \
    } while (0)
#define CELTY_CLOCK() clock64()
#define CELTY_STORE(k, v)                                                     \
    do {                                                                      \
        if (threadIdx.x == 0 && g_celty_trace) g_celty_trace[blockIdx.x * 16 + (k)] = (long long)(v); \
    } while (0)
#else
#define CELTY_MARK(k)
#define CELTY_CLOCK() 0ll
#define CELTY_STORE(k, v)
#endif
#define CELTY_STEPCLK(slot)
#ifdef CELTY_GUARD
#define CELTY_CHECK(ok, code, value)                                                                   \
    ((ok) ? true                                                                                       \
          : (g_celty_trace ? (g_celty_trace[192 * 16 + 2 * (code)] = (long long)(value),               \
                              g_celty_trace[192 * 16 + 2 * (code) + 1] += 1, false)                    \
                           : false))
#else
#define CELTY_CHECK(ok, code, value) true
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

__device__ __forceinline__ uint4 lds128(uint32_t a)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}

__device__ __forceinline__ uint32_t lds32(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}

// One lane's work on a sub-block, as a three-stage software pipeline over the steps q of its run
// stream (a step = one group of 8 entries of every lane that still has one):
//   fetch(q+2)   128-bit value vector + 32-bit run word from the ring slot
//   decode(q)    run-length decode on packed bytes, cell addresses, FP16 -> FP32; the 8 accumulator
//                loads are issued here ...
//   finish(q-1)  ... and consumed one step later: fmaf + store.
// Rows of one lane only grow within a column, so the cells of different steps never coincide and the
// loads of step q may overtake the stores of step q-1.  Lanes that have run out of groups work on the
// spare rows of their bank with zero values, which keeps the loop free of divergent branches.
struct StepBuf {
    uint4 v;            // fetched values
    uint32_t w;         // fetched runs
    bool act;           // this lane has a group in the fetched step
    uint32_t a[8];      // cell addresses of the decoded step
    float c[8];         // accumulator values loaded for the decoded step
    float f[8];         // its 8 weights in FP32
};

__device__ __forceinline__ void step_fetch(StepBuf &b, uint32_t gl, uint32_t q, uint32_t &cum, uint32_t lt_mask,
                                           uint32_t vbase, uint32_t rbase, uint32_t slot_end)
{
    b.act = gl > q;
    const uint32_t bal = __ballot_sync(kFull, b.act);
    const uint32_t k = cum + __popc(bal & lt_mask);
    cum += __popc(bal);
    b.v = make_uint4(0, 0, 0, 0);
    b.w = 0;
    if (b.act && CELTY_CHECK(vbase + 16 * k + 16 <= slot_end && rbase + 4 * k + 4 <= slot_end, 1, k)) {
        b.v = lds128(vbase + 16 * k);
        b.w = lds32(rbase + 4 * k);
    }
    (void)slot_end;
}

__device__ __forceinline__ void step_decode(StepBuf &b, uint32_t &cell, uint32_t spare_cell, uint32_t slab_end)
{
    uint32_t even, odd, total;
    decode_group(b.w, even, odd, total);
    const uint32_t base = b.act ? cell : spare_cell;
    if (b.act) cell += (total + kGroup) * 128u;
    // cell address = base + 128 * offset byte: one dot-product-accumulate per entry
    b.a[0] = __dp4a(even, 0x00000080u, base);
    b.a[1] = __dp4a(odd, 0x00000080u, base);
    b.a[2] = __dp4a(even, 0x00008000u, base);
    b.a[3] = __dp4a(odd, 0x00008000u, base);
    b.a[4] = __dp4a(even, 0x00800000u, base);
    b.a[5] = __dp4a(odd, 0x00800000u, base);
    b.a[6] = __dp4a(even, 0x80000000u, base);
    b.a[7] = __dp4a(odd, 0x80000000u, base);
#pragma unroll
    for (int e = 0; e < 8; ++e)
        if (!CELTY_CHECK(b.a[e] + 4 <= slab_end, 2, b.a[e])) b.a[e] = spare_cell;
    (void)slab_end;
#pragma unroll
    for (int e = 0; e < 8; ++e) asm volatile("ld.shared.f32 %0, [%1];" : "=f"(b.c[e]) : "r"(b.a[e]));
    const float2 f01 = __half22float2(*reinterpret_cast<const __half2 *>(&b.v.x));
    const float2 f23 = __half22float2(*reinterpret_cast<const __half2 *>(&b.v.y));
    const float2 f45 = __half22float2(*reinterpret_cast<const __half2 *>(&b.v.z));
    const float2 f67 = __half22float2(*reinterpret_cast<const __half2 *>(&b.v.w));
    b.f[0] = f01.x; b.f[1] = f01.y; b.f[2] = f23.x; b.f[3] = f23.y;
    b.f[4] = f45.x; b.f[5] = f45.y; b.f[6] = f67.x; b.f[7] = f67.y;
}

__device__ __forceinline__ void step_finish(const StepBuf &b, float xj)
{
#pragma unroll
    for (int e = 0; e < 8; ++e)
        asm volatile("st.shared.f32 [%0], %1;" ::"r"(b.a[e]), "f"(fmaf(b.f[e], xj, b.c[e])) : "memory");
}

// Shared-memory carve-up of the fused kernel, computed by ONE function for the kernel and for the host
// (which sizes the launch with .total), so that the two can never disagree.
struct FusedSmem {
    size_t acc, ring, bars, items, imeta, lane_base, red, keep, total;
};

__host__ __device__ inline FusedSmem fused_smem_layout(int R, int K, int ncw, int D, int slot_bytes, int cap)
{
    FusedSmem l;
    size_t off = 0;
    l.acc = off;       off += (size_t)ncw * (R + kTileSlack) * 32 * 4;   // FP32 accumulators, one slab per streaming warp
    l.ring = off;      off += (size_t)ncw * D * slot_bytes;              // bulk-copy ring slots (multiples of 128 bytes)
    l.bars = off;      off += (size_t)ncw * D * 8;                       // one mbarrier per slot
    l.items = off;     off += (size_t)ncw * cap * 8;                     // {column, x bits} per looked-up item
    l.imeta = off;     off += (size_t)ncw * cap * 8;                     // {offset/16, bytes} of its sub-block
    l.lane_base = off; off += (size_t)ncw * 128;                         // rank of each lane's first survivor
    l.red = off;       off += 32 * 128;                                  // [32 warps][32 lanes] final-sum scratch
    l.keep = off;      off += ((size_t)((K + 31) / 32) * 4 + 15) / 16 * 16;   // one keep bit per activation
    l.total = off;
    return l;
}

__global__ void __launch_bounds__(512, 1) k_spmspv_fused(const FusedParams p)
{
    extern __shared__ __align__(128) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthreads = blockDim.x, nwarps = nthreads >> 5;
    const int slab_words = (p.R + kTileSlack) * 32;
    // The first ncw = G * Sc warps stream columns; the others only help with the phases that are plain
    // data-parallel work (thresholding, clearing, storing and summing partial vectors).
    const int ncw = p.G * p.Sc;
    const bool streams = warp < ncw;
    const int cw = streams ? warp : 0;
    // ---- shared memory carve-up
    const FusedSmem lay = fused_smem_layout(p.R, p.K, ncw, p.D, p.slot_bytes, p.cap);
    float *acc = reinterpret_cast<float *>(smem + lay.acc);
    uint8_t *ring = smem + lay.ring;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + lay.bars);
    int2 *items = reinterpret_cast<int2 *>(smem + lay.items) + (size_t)cw * p.cap;      // [cap] {column, x bits}
    uint2 *imeta = reinterpret_cast<uint2 *>(smem + lay.imeta) + (size_t)cw * p.cap;    // [cap] {offset/16, bytes}
    int *lane_base = reinterpret_cast<int *>(smem + lay.lane_base) + cw * 32;
    float *red = reinterpret_cast<float *>(smem + lay.red);
    uint32_t *kbw = reinterpret_cast<uint32_t *>(smem + lay.keep);

    const int part = blockIdx.x % p.P, kslice = blockIdx.x / p.P, nK = gridDim.x / p.P;
    const int g = cw / p.Sc, sl = cw - g * p.Sc;
    const int s = part * p.Sc + sl;                               // this warp's slab; may be >= S (idle)

    CELTY_MARK(0);
    // The sub-block offsets are needed right after the ranks are known: start pulling the table into L2 now.
    {
        const size_t meta_bytes = ((size_t)p.K * p.S + 1) * 4;
        for (size_t o = (size_t)tid * 128; o < meta_bytes; o += (size_t)nthreads * 128)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const uint8_t *>(p.meta) + o));
    }
    // ---- a1: threshold all of x; byte q of the keep words = keep bits of activations 8q .. 8q+7
    const int ngroups = (p.K + 7) >> 3, nwords = (p.K + 31) >> 5;
    uint8_t *kb = reinterpret_cast<uint8_t *>(kbw);
    for (int q = tid; q < nwords * 4; q += nthreads) {
        uint32_t keep = 0;
        if (q < ngroups) {
            uint32_t h[4];
            if (8 * q + 8 <= p.K && CELTY_CHECK(q >= 0, 5, q)) {
                const uint4 v = __ldg(reinterpret_cast<const uint4 *>(p.x + 8 * q));
                h[0] = v.x; h[1] = v.y; h[2] = v.z; h[3] = v.w;
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t lo = (8 * q + 2 * k < p.K) ? p.x[8 * q + 2 * k] : 0u;
                    const uint32_t hi = (8 * q + 2 * k + 1 < p.K) ? p.x[8 * q + 2 * k + 1] : 0u;
                    h[k] = lo | (hi << 16);
                }
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint16_t bits = (uint16_t)((k & 1) ? (h[k >> 1] >> 16) : (h[k >> 1] & 0xFFFFu));
                const float f = __half2float(__ushort_as_half(bits));
                if (8 * q + k < p.K && !(fabsf(f) <= p.tau)) keep |= 1u << k;
            }
        }
        if (CELTY_CHECK(q < nwords * 4, 6, q)) kb[q] = (uint8_t)keep;
    }
    // clear the accumulators while those loads are in flight
    {
        float4 *acc4 = reinterpret_cast<float4 *>(acc);
        for (int i = tid; i < ncw * slab_words / 4; i += nthreads)
            if (CELTY_CHECK((size_t)i * 16 + 16 <= (size_t)ncw * slab_words * 4, 7, i)) acc4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (lane == 0 && streams) {
        for (int d = 0; d < p.D; ++d) mbar_init(smem_u32(&bars[warp * p.D + d]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    CELTY_MARK(1);

    if (streams) {
        // ---- every streaming warp ranks the survivors by itself: lane L owns keep words [L*c, (L+1)*c)
        const int wpl = (nwords + 31) >> 5;
        const int w0 = min(nwords, lane * wpl), w1 = min(nwords, w0 + wpl);
        int mine = 0;
        for (int w = w0; w < w1; ++w) mine += __popc(kbw[w]);
        int incl = mine;
    #pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int up = __shfl_up_sync(kFull, incl, d);
            if (lane >= d) incl += up;
        }
        const int n = __shfl_sync(kFull, incl, 31);
        lane_base[lane] = incl - mine;
        __syncwarp();
        if (blockIdx.x == 0 && tid == 0) *p.count = n;
        // warp group u of nK * G owns ranks [u*n/units, (u+1)*n/units)
        const int64_t units = (int64_t)nK * p.G, u = (int64_t)kslice * p.G + g;
        const int r_begin = (int)(u * n / units), r_end = (int)((u + 1) * n / units);
        CELTY_MARK(2);

        const uint32_t cell0 = smem_u32(acc + (size_t)warp * slab_words) + 4u * lane;
        const uint32_t spare0 = cell0 + (uint32_t)p.R * 128u;         // first spare row of this lane's bank
        const uint32_t slab_end = cell0 - 4u * lane + (uint32_t)slab_words * 4u;
        const uint32_t ring0 = smem_u32(ring + (size_t)warp * p.D * p.slot_bytes);
        const uint32_t bar0 = smem_u32(&bars[warp * p.D]);
        const uint32_t lt_mask = (1u << lane) - 1u;
        uint32_t issued = 0, consumed = 0;                            // ring positions of this warp
        bool failed = false;
        long long dbg_wait = 0, dbg_comp = 0, dbg_steps = 0;          // development builds only
        (void)dbg_wait; (void)dbg_comp; (void)dbg_steps;

        for (int rb = r_begin; rb < r_end && !failed; rb += p.cap) {
            const int cnt = min(p.cap, r_end - rb);
            // ---- column of rank r: the lane whose words hold it, then the word, then the bit
            for (int i = lane; i < cnt; i += 32) {
                const int r = rb + i;
                int o = 0;
    #pragma unroll
                for (int step = 16; step; step >>= 1)
                    if (lane_base[o + step] <= r) o += step;
                int rem = r - lane_base[o], w = o * wpl;
                for (;;) {
                    if (!CELTY_CHECK(w >= 0 && w < nwords, 8, w)) { w = 0; rem = 0; break; }
                    const int pc = __popc(kbw[w]);
                    if (rem < pc) break;
                    rem -= pc;
                    ++w;
                }
                int j = 32 * w + (int)__fns(kbw[w], 0, rem + 1);
                if (!CELTY_CHECK(j >= 0 && j < p.K && w < nwords, 3, j)) j = 0;
                const uint16_t xb = p.x[j];
                if (CELTY_CHECK(i < p.cap, 9, i)) items[i] = make_int2(j, (int)xb);
                if (part == 0 && sl == 0 && CELTY_CHECK(r >= 0 && r < p.K, 10, r)) {
                    p.idx[r] = j;
                    p.val[r] = xb;
                }
                if (s < p.S) {
                    const uint32_t o0 = p.meta[(size_t)j * p.S + s], o1 = p.meta[(size_t)j * p.S + s + 1];
                    imeta[i] = make_uint2(o0, (o1 - o0) * 16u);
                    if (!CELTY_CHECK(o1 >= o0 && (o1 - o0) * 16u <= (uint32_t)p.slot_bytes && o1 > o0 &&
                                         (long long)o1 * 16 <= p.stream_bytes, 4, o1 - o0))
                        imeta[i] = make_uint2(0u, 32u);
                }
            }
            __syncwarp();
            if (s >= p.S) continue;
            // ---- a2: keep D copies in flight
            auto issue = [&](int i) {
                const uint32_t slot = issued % (uint32_t)p.D;
                const uint2 im = imeta[i];
                mbar_expect_tx(bar0 + 8u * slot, im.y);
                bulk_load(ring0 + slot * (uint32_t)p.slot_bytes, p.stream + (size_t)im.x * 16, im.y, bar0 + 8u * slot);
                ++issued;
            };
            if (lane == 0)
                for (int i = 0; i < min(cnt, p.D); ++i) issue(i);
            CELTY_MARK(3);
            for (int i = 0; i < cnt; ++i) {
                const uint32_t slot = consumed % (uint32_t)p.D, parity = (consumed / (uint32_t)p.D) & 1u;
                const long long t_wait0 = CELTY_CLOCK();
                if (!mbar_wait_bounded(bar0 + 8u * slot, parity)) failed = true;
                const long long t_wait1 = CELTY_CLOCK();
                dbg_wait += t_wait1 - t_wait0;
                failed = __any_sync(kFull, failed);
                if (failed) break;
                if (i == 0) CELTY_MARK(4);
                ++consumed;
                if (i == 0) CELTY_STEPCLK(41);
                const uint32_t sub = ring0 + slot * (uint32_t)p.slot_bytes;
                const float xj = __half2float(__ushort_as_half((uint16_t)items[i].y));
                // ---- a3 + a4: header = groups per lane; vectors are stored step-major, active lanes only
                uint32_t gl;
                asm volatile("ld.shared.u8 %0, [%1];" : "=r"(gl) : "r"(sub + lane));
                const uint32_t steps = __reduce_max_sync(kFull, gl);
                const uint32_t Gs = __reduce_add_sync(kFull, gl);
                const uint32_t vbase = sub + 32, rbase = vbase + 16 * Gs;
                const uint32_t slot_end = sub + (uint32_t)p.slot_bytes;
                if (i == 0) CELTY_STEPCLK(42);
                if (p.flags & 1) {
                    uint32_t cell = cell0, cum = 0;
                    StepBuf b0, b1;
                    step_fetch(b0, gl, 0, cum, lt_mask, vbase, rbase, slot_end);
                    step_fetch(b1, gl, 1, cum, lt_mask, vbase, rbase, slot_end);
                    step_decode(b0, cell, spare0, slab_end);                           // step 0
                    step_fetch(b0, gl, 2, cum, lt_mask, vbase, rbase, slot_end);
                    for (uint32_t q = 1; q <= steps; q += 2) {
                        if (i == 0) CELTY_STEPCLK(q);
                        step_decode(b1, cell, spare0, slab_end);                       // step q
                        step_finish(b0, xj);                                 // step q-1
                        step_fetch(b1, gl, q + 2, cum, lt_mask, vbase, rbase, slot_end);
                        step_decode(b0, cell, spare0, slab_end);                       // step q+1
                        step_finish(b1, xj);                                 // step q
                        step_fetch(b0, gl, q + 3, cum, lt_mask, vbase, rbase, slot_end);
                    }
                } else {
                    // plain loop: vectors of step q+1 are loaded before step q is accumulated
                    uint32_t cell = cell0, cum = 0;
                    StepBuf b0, b1;
                    step_fetch(b0, gl, 0, cum, lt_mask, vbase, rbase, slot_end);
                    for (uint32_t q = 0; q < steps; ++q) {
                        if (i == 0) CELTY_STEPCLK(q);
                        step_fetch(b1, gl, q + 1, cum, lt_mask, vbase, rbase, slot_end);
                        if (b0.act) {
                            step_decode(b0, cell, spare0, slab_end);
                            step_finish(b0, xj);
                        }
                        b0.v = b1.v; b0.w = b1.w; b0.act = b1.act;
                    }
                }
                __syncwarp();
                if (i == 0) CELTY_STEPCLK(40);
                dbg_comp += CELTY_CLOCK() - t_wait1;
                dbg_steps += steps;
                if (lane == 0 && i + p.D < cnt) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    issue(i + p.D);
                }
            }
            issued = __shfl_sync(kFull, issued, 0);
            CELTY_STORE(10, dbg_wait);
            CELTY_STORE(11, dbg_comp);
            CELTY_STORE(12, dbg_steps);
            CELTY_STORE(13, cnt);
        }
        if (failed) {
            // give copies that are still in flight a last (bounded) chance to land before the block exits
            for (; consumed < issued; ++consumed)
                mbar_wait_bounded(bar0 + 8u * (consumed % (uint32_t)p.D), (consumed / (uint32_t)p.D) & 1u);
            if (lane == 0) atomicOr(p.status, kStatusTimeout);
        }
    }
    __syncthreads();
    CELTY_MARK(5);

    // ---- a5, stage 1: add the G accumulators, store the block's partial (accumulator layout, no slack rows)
    const int tile_words = p.R * 32, part_words = p.Sc * tile_words;
    {
        float4 *mine4 = reinterpret_cast<float4 *>(p.partials + (size_t)blockIdx.x * part_words);
        const float4 *acc4 = reinterpret_cast<const float4 *>(acc);
        for (int q4 = tid; q4 < part_words / 4; q4 += nthreads) {
            const int fsl = (q4 * 4) / tile_words, rem = q4 * 4 - fsl * tile_words;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int gg = 0; gg < p.G; ++gg) {
                const size_t ai = ((size_t)(gg * p.Sc + fsl) * slab_words + rem) >> 2;
                if (!CELTY_CHECK(ai * 16 + 16 <= (size_t)ncw * slab_words * 4, 12, ai)) continue;
                const float4 t = acc4[ai];
                v.x += t.x; v.y += t.y; v.z += t.z; v.w += t.w;
            }
            if (CELTY_CHECK(((size_t)blockIdx.x * part_words + (size_t)q4 * 4 + 4) <= (size_t)gridDim.x * part_words, 11, q4))
                __stcg(mine4 + q4, v);
        }
    }
    __syncthreads();
    CELTY_MARK(6);
    if (tid == 0) {
        __threadfence();                                          // the block's stores, ordered by the barrier above
        atomicAdd(&p.tickets[0], 1u);
        bool ok = false;
        for (uint32_t it = 0; it < kSpinLimit; ++it) {
            if (ld_acquire_u32(&p.tickets[0]) >= gridDim.x) { ok = true; break; }
            __nanosleep(32);
        }
        if (!ok) atomicOr(p.status, kStatusTimeout);
    }
    __syncthreads();
    CELTY_MARK(7);

    // ---- a5, stage 2: the nK blocks of a part share its words; partial b of this part = block b*P + part
    {
        const int wpc = (((part_words + nK - 1) / nK) + 31) & ~31;
        const int wb = kslice * wpc, we = min(part_words, wb + wpc);
        for (int chunk = wb; chunk < we; chunk += 32) {
            const int word = chunk + lane;
            float sum = 0.f;
            if (word < we) {
                // up to 8 loads in flight per lane; the order of the additions is fixed
                const float *src = p.partials + (size_t)part * part_words + word;
                const size_t stride = (size_t)p.P * part_words;
                for (int b0 = warp; b0 < nK; b0 += 8 * nwarps) {
                    float t[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int b = b0 + k * nwarps;
                        t[k] = (b < nK && CELTY_CHECK((size_t)(b * p.P + part) * part_words + word <
                                                          (size_t)gridDim.x * part_words, 13, b))
                                   ? __ldcg(src + (size_t)b * stride) : 0.f;
                    }
#pragma unroll
                    for (int k = 0; k < 8; ++k) sum += t[k];
                }
            }
            red[warp * 32 + lane] = sum;
            __syncthreads();
            if (warp == 0 && word < we) {
                float total = 0.f;
                for (int ww = 0; ww < nwarps; ++ww) total += red[ww * 32 + lane];
                const int fsl = word / tile_words, rem = word - fsl * tile_words;
                const int i = rem >> 5, t = 32 * (part * p.Sc + fsl) + (rem & 31), row = t * p.R + i;
                if (t < p.T && row < p.M && CELTY_CHECK(row >= 0, 14, row)) p.y[row] = total;
            }
            __syncthreads();
        }
    }
    CELTY_MARK(8);
    if (tid == 0) {
        const uint32_t t = atomicAdd(&p.tickets[1], 1u);
        if (t == gridDim.x - 1) {                                  // last one out resets both tickets
            atomicExch(&p.tickets[0], 0u);
            atomicExch(&p.tickets[1], 0u);
        }
    }
    CELTY_MARK(9);
}

struct FusedPlan {
    int G, Sc, P, D, slot_bytes, cap, threads, grid;
    size_t smem;
};

inline size_t fused_smem_bytes(int R, int K, int G, int Sc, int D, int slot_bytes, int cap)
{
    return fused_smem_layout(R, K, G * Sc, D, slot_bytes, cap).total;
}
