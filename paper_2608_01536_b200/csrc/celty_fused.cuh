// The single-launch SpMSpV kernel for the LANE_TILE layout (included by celty_kernels.cu inside its
// anonymous namespace, after decode_group).
//
// One launch does the whole call (Sections 3.1-3.3):
//   a0  the last warp of every block clears its share of y and takes a ticket (the merge at the end adds into y);
//   a1  every block thresholds all of x (K <= a few 10k values, served by L2) into one keep bit per
//       activation and ranks the survivors (popcounts + warp scans); each warp team then looks up the
//       columns whose ranks belong to it -- the list is balanced over all teams by count -- and their
//       sub-block offsets, which it finds in a window of the offset table that the block copied into
//       shared memory when it started.  The team that owns a rank on slab 0 also writes it to the global
//       list (index, value, count) for the API;
//   a2  each team streams the sub-blocks (column j, slab s) of its columns from HBM into its ring of
//       shared-memory slots with bulk asynchronous copies (cp.async.bulk + mbarrier complete_tx), D deep;
//   a3  each lane decodes its own tile's runs on packed bytes and keeps a running row;
//   a4  value * x_j is accumulated (FP16 x FP16 + FP32 fused multiply-add) into the lane's private bank of
//       the team's accumulator;
//   a5  the block adds its G accumulators; the row map makes a slab's accumulator a sequence of 32*C-row
//       segments of y, and each goes out as one bulk reduce-add copy (FP32 add in L2) once the tickets show
//       that every block has cleared its share of y.  Options: clusters of 2 or 4 thread blocks that first add
//       their sums through distributed shared memory, each block then sending only the segments it owns
//       (measured: no faster, so off by default); per-block partial vectors, a bounded grid-wide ticket
//       barrier and a sum in a fixed order (bit-reproducible, no clearing of y).
//   then, on request: an FP16 copy of y, or SiLU(gate) * up of a stacked [gate; up] product with its
//       thresholded list (fused_epilogue), once a second ticket shows that every block's adds are done.
//
// Rows are split over P parts of Sc slabs each, columns over the blocks of a part and, inside a block, over
// G teams per slab; a team = one warp (or, with pp, two warps that take turns) with its own accumulator slab.
// Blocks that are left over when the grid does not divide by P may serve several parts each with fewer teams per
// part (FusedParams::mix).  Every block must be resident at once (grid <= SM count) because of the tickets.  All
// waits are bounded: when one runs out the kernel sets kStatusTimeout in the status word and carries on to a clean
// exit.

// Shared-memory carve-up of the fused kernel, computed by ONE function for the kernel and for the host
// (which sizes the launch with .total), so that the two can never disagree.
struct FusedSmem {
    size_t acc, ring, bars, flag, items, imeta, zero, keep, wrel, blk, blkw, total;
};

__host__ __device__ inline FusedSmem fused_smem_layout(int R, int K, int teams, int D, int slot_bytes, int cap)
{
    FusedSmem l;
    uint32_t off = 0;
    l.acc = off;       off += (uint32_t)teams * (R + kTileSlack) * 32 * 4;   // FP32 accumulators, one slab per team
    l.ring = off;      off += (uint32_t)teams * D * slot_bytes;              // bulk-copy ring slots (multiples of 128 bytes)
    l.bars = off;      off += (uint32_t)teams * D * 8 + 8;                   // one "full" mbarrier per slot, one for the offset window
    l.flag = off;      off += (uint32_t)teams * 4;                           // per team: a wait of one of its warps ran out
    off = (off + 15) / 16 * 16;
    l.items = off;     off += (uint32_t)teams * cap * 8;                     // {column, x bits} per looked-up item
    l.imeta = off;     off += (uint32_t)teams * cap * 8;                     // {offset/16, bytes} of its sub-block
    l.zero = off;      off += 16;                                          // the all-zero group that idle lanes fetch
    l.keep = off;      off += ((uint32_t)((K + 31) / 32) * 4 + 15) / 16 * 16;   // one keep bit per activation
    l.wrel = off;      off += ((uint32_t)((K + 31) / 32) * 4 + 15) / 16 * 16;   // survivors before each keep word, in its block of 32
    l.blk = off;       off += ((uint32_t)((K + 1023) / 1024) * 4 + 15) / 16 * 16; // survivors in each block of 32 keep words
    l.blkw = off;      off += 16 * (((uint32_t)((K + 1023) / 1024) * 4 + 15) / 16 * 16);   // per warp: survivors before each block
    l.total = off;
    return l;
}

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
    uint32_t *tickets;         // [0] y cleared / partial stored, [1] adds done (work after the merge) / departed
    float *partials;           // gridDim.x vectors of Sc * R * 32 floats (accumulator layout)
    int M, K, R, S, C;         // rows, columns, local rows per tile, slabs, chunk of the row map (tile_row)
    int G, Sc, P, D;           // teams per slab, slabs per block, row parts, ring depth
    int cl;                    // thread blocks per cluster (1, 2 or 4); blocks of a cluster share a row part
    int pp;                    // 1: two warps per team that take turns at the team's accumulator (see the kernel)
    // mix >= 2 (bulk reduce-add merge without clusters): the gridDim mod P blocks that are left when every row part
    // has floor(gridDim / P) blocks are not given to the first parts (which would then finish early, one slice
    // ahead of the others); each of them serves mix = P / (gridDim mod P) consecutive parts instead, with G / mix
    // teams per slab, so that every part is shared by the same number of teams.  units_inv then holds
    // floor(2^32 / (floor(gridDim / P) * G + G / mix)).
    int mix;
    int slot_bytes;            // ring slot size, multiple of 128
    int cap;                   // columns a team looks up per batch
    int win_cols;              // columns of the offset table a block copies into shared memory at its start
    FusedSmem lay;             // the block's shared memory, worked out once on the host (fused_smem_layout)
    int clear_rows, clear_extra;   // M / gridDim.x and M mod gridDim.x: block b clears clear_rows (+ 1 if b < clear_extra) rows of y
    // teams that share the survivor list of a row part: units = (column slices of the part) * G;
    // units_inv = floor(2^32 / units) for parts with gridDim / cl / P clusters, units_inv_long for those with
    // one cluster more
    uint32_t units_inv, units_inv_long;
    int merge;                 // 0: partial vectors + ordered final sum; 1: bulk reduce-add of row segments into y
    uint32_t spin_limit;       // polls a bounded wait makes before it gives up
    // a1 done by the producer of the activations: when list_count is not null the surviving columns and their
    // values come from this list (any order, every column at most once) and x and tau are not looked at
    const int32_t *list_idx;
    const uint16_t *list_val;
    const int32_t *list_count;
    // The activations are not given but made on the fly from the FP32 result of a stacked [gate; up] product
    // (2K values, gate first): x_j = SiLU(g_j) * u_j rounded to FP16, for the down projection.  h_out (may be
    // null) receives the K FP16 values.
    const float *swiglu_in;
    uint16_t *h_out;
    // Work on y after the merge (bulk reduce-add merge only): 0 none; 1 an FP16 copy of y; 2 y holds a stacked
    // [gate; up] product of 2I rows: h_i = SiLU(y_i) * y_{I+i} rounded to FP16, stored, and the (i, h_i) with
    // |h_i| > ep_tau appended to a list that the next product takes as its survivors
    int ep_kind;
    uint16_t *ep_out;
    float ep_tau;
    int32_t *ep_idx;
    uint16_t *ep_val;
    int32_t *ep_count;
};

constexpr uint32_t kSpinLimit = 1u << 21;   // default for FusedParams::spin_limit

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
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

// a / b for 0 <= a < 2^20 and b > 0 through one approximate float division.  Exact for such operands: (a + 0.5) / b
// is at least 0.5 / b away from every integer, and the division's error (2 units in the last place of a value of
// at most a / b) stays below 2^-22 a / b, which is less than that for a < 2^21.  The block and team indices of the
// kernel are made of a dozen such quotients, and an integer division is 25 instructions of code that a block runs
// once.
__device__ __forceinline__ int idiv_small(int a, int b)
{
    return (int)__fdividef((float)a + 0.5f, (float)b);
}

// Wait for a phase of an mbarrier with an iteration limit; false = gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit)
{
#pragma unroll 1
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > 256) __nanosleep(128);
    }
    return false;
}

// Bulk asynchronous copy global -> shared (1-D, no tensor map; every sub-block has exactly one consumer,
// the team that asked for it); src, dst and bytes are multiples of 16.  Every lane of a converged warp calls
// this; one elected lane announces the bytes on the mbarrier and issues the copy, both under a predicate
// (no branch); completion is signalled on the mbarrier as transferred bytes.
__device__ __forceinline__ void bulk_load_elected(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile(
        "{\n\t.reg .pred P;\n\t"
        "elect.sync _|P, 0xffffffff;\n\t"
        "@P mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n\t"
        "@P cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%2], [%3], %1, [%0];\n\t}" ::"r"(bar),
        "r"(bytes), "r"(dst), "l"(src)
        : "memory");
}

// Barrier across the thread blocks of the cluster (release / acquire: shared-memory writes made before it
// are visible to the other blocks' distributed-shared-memory reads after it).
__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// 128-bit load from the shared memory of block `rank` of the cluster, at this block's address `local`.
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t local, uint32_t rank)
{
    uint32_t remote;
    float4 v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "r"(remote)
                 : "memory");
    return v;
}

// Polling load that goes to L2 every time but carries no ordering (and so leaves the L1 of the other
// warps alone); the caller fences once after the value it waits for has shown up.
__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// One lane's work on the steps of a sub-block, as a three-stage software pipeline (a step =
// one group of 8 entries of every lane that still has one):
//   fetch(q+2)   128-bit value vector + 32-bit run word from the ring slot
//   decode(q)    run-length decode on packed bytes, cell addresses; the 8 accumulator loads are
//                issued here ...
//   finish(q-1)  ... and consumed one step later: multiply-add + store.
// Rows of one lane only grow within a column, so the cells of different steps never coincide and the
// loads of step q may overtake the stores of step q-1.
// Nothing is predicated: a lane without a group in a step fetches an all-zero group (zero values, zero
// runs) from a zero block instead and adds 0 to the 8 spare rows at the end of its tile (its own bank;
// no real entry lives there, so it does not matter who else does the same at the same time).  Such a
// lane has no group in any later step of the item either, so its running row is dead from then on.
struct StepBuf {
    uint4 v;            // fetched values
    uint32_t w;         // fetched runs
    bool act;           // this lane has a group in the fetched step
    uint32_t a[8];      // cell addresses of the decoded step
    float c[8];         // accumulator values loaded for the decoded step
    uint4 h;            // its 8 weights (FP16 pairs)
};

__device__ __forceinline__ float lds_f32(uint32_t a)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(a));
    return v;
}

__device__ __forceinline__ void sts_f32(uint32_t a, float v)
{
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(a), "f"(v) : "memory");
}

// d = a * x + c with FP16 a (both halves of `pair`) and x, FP32 c and d: the product of two FP16 numbers
// is exact in FP32, so this rounds once, exactly like converting to FP32 and calling fmaf.
__device__ __forceinline__ void fma_pair(uint32_t pair, uint16_t x, float c0, float c1, float &d0, float &d1)
{
    asm("{\n\t.reg .b16 lo, hi;\n\t"
        "mov.b32 {lo, hi}, %2;\n\t"
        "fma.rn.f32.f16 %0, lo, %3, %4;\n\t"
        "fma.rn.f32.f16 %1, hi, %3, %5;\n\t}"
        : "=f"(d0), "=f"(d1)
        : "r"(pair), "h"(x), "f"(c0), "f"(c1));
}

__device__ __forceinline__ void step_fetch(StepBuf &b, uint32_t gl, uint32_t q, uint32_t q_end, uint32_t &cum,
                                           uint32_t lt_mask, uint32_t vbase, uint32_t rbase, uint32_t zeros)
{
    bool act = gl > q && q < q_end;
    const uint32_t bal = __ballot_sync(kFull, act);
    const uint32_t k = cum + __popc(bal & lt_mask);
    cum += __popc(bal);
    b.act = act;
    const uint32_t va = act ? vbase + 16 * k : zeros, ra = act ? rbase + 4 * k : zeros;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(b.v.x), "=r"(b.v.y), "=r"(b.v.z), "=r"(b.v.w) : "r"(va));
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(b.w) : "r"(ra));
}

// kRegRows > 0 (the register-accumulation study): cells below `reg_lim` belong to the lane's first kRegRows local
// rows, whose sums live in registers; for them the accumulator is not loaded (the product alone is stored, and
// collected after the sub-block), which is what takes shared-memory loads out of the loop.
template <int kRegRows>
__device__ __forceinline__ void step_decode(StepBuf &b, uint32_t &cell, uint32_t spare, uint32_t reg_lim)
{
    uint32_t even, odd, total;
    decode_group(b.w, even, odd, total);
    cell = b.act ? cell : spare;
    // cell address = cell + 128 * offset byte: one dot-product-accumulate per entry (measured faster on
    // B200 than a byte permute followed by a multiply-add)
    b.a[0] = __dp4a(even, 0x00000080u, cell);
    b.a[1] = __dp4a(odd, 0x00000080u, cell);
    b.a[2] = __dp4a(even, 0x00008000u, cell);
    b.a[3] = __dp4a(odd, 0x00008000u, cell);
    b.a[4] = __dp4a(even, 0x00800000u, cell);
    b.a[5] = __dp4a(odd, 0x00800000u, cell);
    b.a[6] = __dp4a(even, 0x80000000u, cell);
    b.a[7] = __dp4a(odd, 0x80000000u, cell);
    b.h = b.v;
    cell += (total + kGroup) * 128u;
#pragma unroll
    for (int e = 0; e < 8; ++e) b.c[e] = (kRegRows > 0 && b.a[e] < reg_lim) ? 0.f : lds_f32(b.a[e]);
    (void)reg_lim;
}

__device__ __forceinline__ void step_finish(const StepBuf &b, uint16_t xj)
{
    float d[8];
    fma_pair(b.h.x, xj, b.c[0], b.c[1], d[0], d[1]);
    fma_pair(b.h.y, xj, b.c[2], b.c[3], d[2], d[3]);
    fma_pair(b.h.z, xj, b.c[4], b.c[5], d[4], d[5]);
    fma_pair(b.h.w, xj, b.c[6], b.c[7], d[6], d[7]);
#pragma unroll
    for (int e = 0; e < 8; ++e) sts_f32(b.a[e], d[e]);
}

// Work on the finished y (FusedParams::ep_kind), every block on an equal share of the rows.  A function of its own
// (not inlined), so that what it needs in registers does not weigh on the streaming loop of the kernel.
// SiLU(gate) * up evaluated in FP32 and rounded once to FP16 (bit pattern): the one formula behind the work after
// a gate/up product and behind the down projection that makes its activations on the fly.
__device__ __forceinline__ uint32_t swiglu_half_bits(float gate, float up)
{
    return (uint32_t)__half_as_ushort(__float2half_rn(gate / (1.f + expf(-gate)) * up));
}

// The group of 8 activations that the end of x cuts short (K not a multiple of 8), zero-filled.  Out of line: one
// thread of a block needs it, if any, and the thresholding pass is unrolled four times around the call.
__device__ __noinline__ uint4 ragged_group(const uint16_t *x, int K, int q)
{
    uint32_t h[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t lo = (8 * q + 2 * k < K) ? x[8 * q + 2 * k] : 0u;
        const uint32_t hi = (8 * q + 2 * k + 1 < K) ? x[8 * q + 2 * k + 1] : 0u;
        h[k] = lo | (hi << 16);
    }
    return make_uint4(h[0], h[1], h[2], h[3]);
}

struct EpilogueArgs {
    const float *y;
    uint32_t *tickets, *status;
    uint32_t spin_limit;
    int M, ep_kind;
    uint16_t *ep_out;
    float ep_tau;
    int32_t *ep_idx;
    uint16_t *ep_val;
    int32_t *ep_count;
};

__device__ __noinline__ void fused_epilogue(const EpilogueArgs p)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthreads = blockDim.x, nwarps = nthreads >> 5;
    // ---- work on the finished y.  This block's adds must have been performed (not merely read out of shared
    // memory), then every block's: a second wrap-around ticket, as for the clearing of y.
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    __threadfence();
    __syncthreads();
    __shared__ int ep_warp[17];
    if (tid == 0) {
        __threadfence();
        const uint32_t t = atomicInc(&p.tickets[1], 2u * gridDim.x - 1u);
        const bool low_half = t < gridDim.x;
        bool ok = false;
        for (uint32_t it = 0; it < p.spin_limit; ++it) {
            const uint32_t cur = ld_relaxed_u32(&p.tickets[1]);
            if (low_half ? (cur >= gridDim.x) : (cur < gridDim.x)) { ok = true; break; }
            __nanosleep(64);
        }
        __threadfence();
        if (!ok) atomicOr(p.status, kStatusTimeout);
    }
    __syncthreads();
    // every block takes an equal share of the rows; y is read past L1 (it was written by adds in L2)
    if (p.ep_kind == 1) {
        // (shares without a 64-bit division: n / blocks rows each, the first n mod blocks one more)
        const int per = p.M / (int)gridDim.x, extra = p.M - per * (int)gridDim.x, b = (int)blockIdx.x;
        const int r0 = b * per + min(b, extra), r1 = r0 + per + (b < extra ? 1 : 0);
        for (int i = r0 + tid; i < r1; i += nthreads) p.ep_out[i] = __half_as_ushort(__float2half_rn(__ldcg(p.y + i)));
        return;
    }
    const int half_rows = p.M / 2;
    const int per = half_rows / (int)gridDim.x, extra = half_rows - per * (int)gridDim.x, b = (int)blockIdx.x;
    const int r0 = b * per + min(b, extra), r1 = r0 + per + (b < extra ? 1 : 0);
    for (int base = r0; base < r1; base += nthreads) {          // the same trip count for every thread
        const int i = base + tid;
        bool keep = false;
        uint16_t hb = 0;
        if (i < r1) {
            const float gt = __ldcg(p.y + i), up = __ldcg(p.y + half_rows + i);
            const __half h = __float2half_rn(gt / (1.f + expf(-gt)) * up);       // SiLU(gate) * up, one FP16 value
            hb = __half_as_ushort(h);
            p.ep_out[i] = hb;
            keep = !(fabsf(__half2float(h)) <= p.ep_tau);                       // the comparator of a1
        }
        // positions in the list: within the warp by ballot, across the warps by a small scan, across the blocks
        // by one atomic add per block and pass (the list comes out in no particular order)
        const uint32_t bal = __ballot_sync(kFull, keep);
        if (lane == 0) ep_warp[warp] = __popc(bal);
        __syncthreads();
        if (tid == 0) {
            int total = 0;
            for (int w = 0; w < nwarps; ++w) {
                const int c = ep_warp[w];
                ep_warp[w] = total;
                total += c;
            }
            ep_warp[16] = total ? atomicAdd(p.ep_count, total) : 0;
        }
        __syncthreads();
        if (keep) {
            const int pos = ep_warp[16] + ep_warp[warp] + __popc(bal & ((1u << lane) - 1u));
            p.ep_idx[pos] = i;
            p.ep_val[pos] = hb;
        }
        __syncthreads();
    }
}

// kExtras = false compiles the list input and the work after the merge out: the plain product keeps its
// register budget (92 registers against 128 with them), which the streaming loop's scheduling depends on.
// kRegRows > 0 is the software analogue of register-file accumulation (Section 4.1, the register / shared-memory
// split of Section 6.4): the first kRegRows local rows of every lane are summed in registers across the team's
// columns and written to the accumulator slab once, at the end.  Those builds run 256 threads per block (eight
// teams at most), which is what leaves a thread room for up to 128 more registers.
// kLean > 0 are the builds for the library's default launch (bulk reduce-add merge, no clusters; 1: one warp per
// team, 2: warp pairs): the code of the options they do not have is not merely skipped but absent.  A block runs
// most of this kernel's code once per call, from an instruction cache that a call's worth of code overflows, so a
// taken branch over code that is not run costs a trip to L2 (250 cycles and more, measured with stand-alone loops:
// a cliff at about 24 KB of code touched per launch); what falls through in sequence is prefetched and costs
// nothing.
template <bool kExtras, int kRegRows, int kLean = 0>
__global__ void __launch_bounds__(kRegRows > 0 ? 256 : 512, 1) k_spmspv_fused(const FusedParams p)
{
    const int pp = kLean ? (kLean == 2 ? 1 : 0) : p.pp;
    const int merge = kLean ? 1 : p.merge;
    const int cl = kLean ? 1 : p.cl;
    extern __shared__ __align__(128) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, nthreads = blockDim.x, nwarps = nthreads >> 5;
    // the warp index through a shuffle: the compiler then knows that it (and every team, slab and loop bound
    // derived from it) is the same for all lanes, and keeps the streaming loop free of divergence handling
    const int warp = __shfl_sync(kFull, tid >> 5, 0);
    const int slab_words = (p.R + kTileSlack) * 32;
    // Warps [0, teams) stream columns, one warp per team; the others only help with the phases that
    // are plain data-parallel work (thresholding, clearing, storing and summing partial vectors).
    // With pp two warps share a team: warp `team` and warp `teams + team`.  Each streams every other column of the
    // team's share into ring slots of its own, and the two take turns at the team's accumulator: while one runs
    // its step loop, the other waits for its next sub-block, reads the header and fetches the first groups, so the
    // accumulator never sits idle through those latencies.  A named barrier per team hands the accumulator over.
    const int teams = p.G * p.Sc;
    // (The partner of warp t is warp t + 8: the two sit on the same warp scheduler, which suits them, since only
    // one of them is in its step loop at any time.)
    const bool streams = pp ? (warp & 7) < teams : warp < teams;
    const int team = streams ? (pp ? (warp & 7) : warp) : 0;
    const int half = streams && pp ? warp >> 3 : 0;               // which of the team's two warps (0 without pp)
    const int stride = 1 + pp, Dw = p.D / stride;                 // columns between a warp's own, ring slots per warp
    const FusedSmem &lay = p.lay;
    float *acc = reinterpret_cast<float *>(smem + lay.acc);
    uint8_t *ring = smem + lay.ring;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + lay.bars);
    int2 *items = reinterpret_cast<int2 *>(smem + lay.items) + (size_t)team * p.cap;      // [cap] {column, x bits}
    uint2 *imeta = reinterpret_cast<uint2 *>(smem + lay.imeta) + (size_t)team * p.cap;    // [cap] {offset/16, bytes}
    int *zero_group = reinterpret_cast<int *>(smem + lay.zero);                           // 16 bytes of zeros
    int *wrel = reinterpret_cast<int *>(smem + lay.wrel);                                 // [nwords]
    const int *blk = reinterpret_cast<const int *>(smem + lay.blk);                       // [nwords / 32] counts
    int *myblk = reinterpret_cast<int *>(smem + lay.blkw) + (size_t)warp * ((lay.blkw - lay.blk) / 4);   // this warp's prefix
    uint32_t *kbw = reinterpret_cast<uint32_t *>(smem + lay.keep);

    // Row part and column slice of this block.  The blocks of a cluster work on the same row part (they add
    // their accumulators before anything goes to y).  The number of clusters need not be a multiple of P: the
    // first (clusters mod P) parts then have one cluster more than the others.
    const int cl_shift = cl >> 1;                                   // cl is 1, 2 or 4
    const int crank = blockIdx.x & (cl - 1), cid = blockIdx.x >> cl_shift, nclusters = gridDim.x >> cl_shift;
    const int cpart = idiv_small(cid, p.P), clusters_per_part = idiv_small(nclusters, p.P);
    int part = cid - cpart * p.P;
    const bool long_part = p.mix < 2 && part < nclusters - clusters_per_part * p.P;
    const int nK = cl * (clusters_per_part + (long_part ? 1 : 0));
    const int kslice = cpart * cl + crank;
    // G teams per slab and Sc slabs in this block; unit0 = this block's first team among the `units` teams that
    // share the survivor list of its part(s)
    int G = p.G, Sc = p.Sc, unit0 = kslice * p.G, units = nK * p.G;
    if (p.mix >= 2) {
        const int nfull = clusters_per_part;                      // (no clusters with mix)
        units = nfull * p.G + idiv_small(p.G, p.mix);
        if ((int)blockIdx.x >= nfull * p.P) {                     // one of the blocks that serve several parts
            G = idiv_small(p.G, p.mix);
            Sc = p.Sc * p.mix;
            part = (int)blockIdx.x - nfull * p.P;                 // counted in groups of mix parts
            unit0 = nfull * p.G;
        }
    }
    const int g = idiv_small(team, Sc), sl = team - g * Sc;
    const int s = part * Sc + sl;                                 // this team's slab; may be >= S (idle)

    // Programmatic dependent launch: let the next kernel of the stream be scheduled as this one's blocks retire,
    // and do everything that touches neither the caller's vectors nor the workspace (warming L2 with the offset
    // table, setting up shared memory) before waiting for the previous kernel of the stream to be complete.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // The sub-block offsets are needed right after the ranks are known.  A block's columns lie around the same
    // fraction of K as its position among the blocks of its row part, so it copies that window of the offset
    // table into shared memory now -- into the accumulator area, which is not in use until the first copies of
    // the entry stream are under way -- and looks there first (columns outside the window: global memory).
    const uint32_t win_bar = smem_u32(&bars[teams * p.D]);
    const uint32_t *win = reinterpret_cast<const uint32_t *>(smem + lay.acc);
    int win_w0 = 0, win_n = 0;                                     // first table word in the window, words in it
    if (p.win_cols > 0) {
        // the middle of the block's share of the columns, if the survivors were spread evenly (a float will do)
        const int mid = (int)((float)(2 * unit0 + G) * (float)p.K / (float)(2 * units));
        const int c0 = max(0, min(p.K - p.win_cols, mid - p.win_cols / 2));
        win_w0 = (c0 * p.S) & ~3;
        win_n = min(((c0 + p.win_cols) * p.S + 1 - win_w0 + 3) & ~3, ((p.K * p.S + 1 + 3) & ~3) - win_w0);
        // (by the first lane of the last warp, which is not a streaming warp unless all are: the first lanes of the
        // streaming warps have their ring barriers to set up at the same time)
        if (tid == nthreads - 32) {
            mbar_init(win_bar, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(win_bar), "r"((uint32_t)win_n * 4u) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                             smem_u32(win)),
                         "l"(p.meta + win_w0), "r"((uint32_t)win_n * 4u), "r"(win_bar)
                         : "memory");
        }
    }
    if (tid < 4) zero_group[tid] = 0;
    if (tid < teams) reinterpret_cast<int *>(smem + lay.flag)[tid] = 0;
    if (streams && lane == 0) {
#pragma unroll 1
        for (int d = 0; d < Dw; ++d) mbar_init(smem_u32(&bars[team * p.D + half * Dw + d]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    uint32_t y_ticket = 0;
    // Bulk reduce-add merge: the adds at the end need a cleared y.  The last warp clears this block's share
    // and announces it right away, so that the fence and the ticket overlap the loads of a1.
    if (merge == 1 && warp == nwarps - 1) {
        const int b = (int)blockIdx.x;
        const int r0 = b * p.clear_rows + min(b, p.clear_extra), r1 = r0 + p.clear_rows + (b < p.clear_extra ? 1 : 0);
#pragma unroll 1
        for (int i = r0 + lane; i < r1; i += 32) p.y[i] = 0.f;
        if (kExtras && p.ep_kind == 2 && blockIdx.x == 0 && lane == 0) *p.ep_count = 0;   // appended to after the merge
        __syncwarp();
        if (lane == 0) {
            __threadfence();
            // The ticket counts modulo 2 * gridDim.x, so it never has to be reset: calls alternate between
            // waiting for the lower and for the upper half.
            y_ticket = atomicInc(&p.tickets[0], 2u * gridDim.x - 1u);
        }
    }
    // ---- a1: threshold all of x.  A thread takes 32 activations (four 128-bit loads) and makes one keep word,
    // and the warp scans the survivor counts of its block of 32 words:
    //   kbw[w]  keep bits of activations 32w .. 32w+31,
    //   wrel[w] survivors in the words before w of the same block of 32 words,
    //   blk[e]  survivors in block e (turned into survivors before block e by the scan below).
    // |x| > tau in FP32 is the same decision as |x| > (tau rounded down to FP16) in FP16; NaN is kept.
    const int ngroups = (p.K + 7) >> 3, nwords = (p.K + 31) >> 5, nblk = (nwords + 31) >> 5;
    const bool from_list = kExtras && p.list_count != nullptr;    // a1 was done by whoever produced the activations
    if (!from_list) {
        const __half2 tau2 = __half2half2(__float2half_rd(p.tau));
#pragma unroll 1
        for (int w0 = 0; w0 < nwords; w0 += nthreads) {             // the same trip count for every thread
            const int w = w0 + tid;
            uint32_t word = 0;
            if (w < nwords) {
                uint32_t h[4][4];
#pragma unroll
                for (int c = 0; c < 4; ++c) {                          // four independent 128-bit loads per thread
                    const int q = 4 * w + c;
                    h[c][0] = h[c][1] = h[c][2] = h[c][3] = 0u;        // zero past the end of x: never kept (tau >= 0)
                    if (kExtras && p.swiglu_in) {                      // the activations are made here, from FP32 gate / up
                        if (q < ngroups) {
                            float gt[8], up[8];
                            if (8 * q + 8 <= p.K && (p.K & 3) == 0) {  // 128-bit loads (the up half starts 16-byte aligned)
                                const float4 a0 = __ldg(reinterpret_cast<const float4 *>(p.swiglu_in + 8 * q));
                                const float4 a1 = __ldg(reinterpret_cast<const float4 *>(p.swiglu_in + 8 * q + 4));
                                const float4 b0 = __ldg(reinterpret_cast<const float4 *>(p.swiglu_in + p.K + 8 * q));
                                const float4 b1 = __ldg(reinterpret_cast<const float4 *>(p.swiglu_in + p.K + 8 * q + 4));
                                gt[0] = a0.x; gt[1] = a0.y; gt[2] = a0.z; gt[3] = a0.w; gt[4] = a1.x; gt[5] = a1.y; gt[6] = a1.z; gt[7] = a1.w;
                                up[0] = b0.x; up[1] = b0.y; up[2] = b0.z; up[3] = b0.w; up[4] = b1.x; up[5] = b1.y; up[6] = b1.z; up[7] = b1.w;
                            } else {
#pragma unroll
                                for (int k = 0; k < 8; ++k) {
                                    const int j = 8 * q + k;
                                    gt[k] = j < p.K ? __ldg(p.swiglu_in + j) : 0.f;          // SiLU(0) * 0 = 0: never kept
                                    up[k] = j < p.K ? __ldg(p.swiglu_in + p.K + j) : 0.f;
                                }
                            }
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const uint32_t lo = swiglu_half_bits(gt[2 * k], up[2 * k]), hi = swiglu_half_bits(gt[2 * k + 1], up[2 * k + 1]);
                                h[c][k] = lo | (hi << 16);
                                // every block makes all of h; the blocks share the writing of it
                                if (p.h_out && (q % gridDim.x) == blockIdx.x) {
                                    if (8 * q + 2 * k < p.K) p.h_out[8 * q + 2 * k] = (uint16_t)lo;
                                    if (8 * q + 2 * k + 1 < p.K) p.h_out[8 * q + 2 * k + 1] = (uint16_t)hi;
                                }
                            }
                        }
                    } else if (8 * q + 8 <= p.K) {
                        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(p.x + 8 * q));
                        h[c][0] = v.x; h[c][1] = v.y; h[c][2] = v.z; h[c][3] = v.w;
                    } else if (__builtin_expect(q < ngroups, 0)) {
                        const uint4 v = ragged_group(p.x, p.K, q);     // the one group that K cuts short
                        h[c][0] = v.x; h[c][1] = v.y; h[c][2] = v.z; h[c][3] = v.w;
                    }
                }
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        // 0xFFFF in a half where |x| <= tau (false for NaN); the keep bits are the complement
                        const uint32_t le = __hle2_mask(__habs2(*reinterpret_cast<const __half2 *>(&h[c][k])), tau2);
                        word |= ((~le & 1u) | ((~le >> 15) & 2u)) << (8 * c + 2 * k);
                    }
                if (32 * w + 32 > p.K) word &= (32 * w < p.K) ? (0xFFFFFFFFu >> (32 * w + 32 - p.K)) : 0u;
            }
            const int cnt = __popc(word);
            int incl = cnt;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {                         // scan within the block of 32 words
                const int up = __shfl_up_sync(kFull, incl, d);
                if (lane >= d) incl += up;
            }
            if (w < nwords) {
                kbw[w] = word;
                wrel[w] = incl - cnt;
            }
            if (lane == 31 && (w >> 5) < nblk) const_cast<int *>(blk)[w >> 5] = incl;
        }
    }
    __syncthreads();
    bool failed = false;
    // the window has had the whole thresholding pass to arrive; nobody may clear an accumulator before it has
    if (p.win_cols > 0 && !mbar_wait_bounded(win_bar, 0, p.spin_limit)) failed = true;
    if (pp) failed = __syncthreads_or(failed);                  // the two warps of a team must agree on what follows
    if (failed) win_n = 0;
    // ---- ranks: every streaming warp turns the block counts into survivors before each block for itself, 32
    // blocks at a time (a copy per warp costs a few hundred bytes and saves a block-wide barrier behind a single
    // warp); the list is then cut into equal shares for the groups that work on different columns.
    int n_surv = 0;
    if (from_list) {
        n_surv = max(0, min(p.K, __ldcg(p.list_count)));
        if (blockIdx.x == 0 && tid == 0) *p.count = n_surv;
    } else if (streams) {
        int carry = 0;
#pragma unroll 1
        for (int e0 = 0; e0 < nblk; e0 += 32) {
            const int e = e0 + lane, cnt = e < nblk ? blk[e] : 0;
            int incl = cnt;
            const int nscan = min(32, nblk - e0);                     // no more steps than there are blocks
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                if (d >= nscan) break;
                const int up = __shfl_up_sync(kFull, incl, d);
                if (lane >= d) incl += up;
            }
            if (e < nblk) myblk[e] = carry + incl - cnt;
            carry += __shfl_sync(kFull, incl, min(31, nblk - e0 - 1));   // the last block's inclusive sum
        }
        __syncwarp();
        n_surv = carry;
        if (blockIdx.x == 0 && warp == 0 && lane == 0) *p.count = carry;
    }

    if (streams) {
        // team u of nK * G owns n / units ranks, the first n mod units teams one more.  n / units without a
        // division: units_inv = floor(2^32 / units) gives a quotient that is at most one too small
        const uint32_t units_inv = long_part ? p.units_inv_long : p.units_inv;
        uint32_t share = __umulhi((uint32_t)n_surv, units_inv), extra = (uint32_t)n_surv - share * (uint32_t)units;
        if (extra >= (uint32_t)units) { ++share; extra -= (uint32_t)units; }
        const int u = unit0 + g;
        const int r_begin = u * (int)share + min(u, (int)extra), r_end = r_begin + (int)share + (u < (int)extra ? 1 : 0);
        const uint32_t slab0 = smem_u32(acc + (size_t)team * slab_words);
        const uint32_t cell0 = slab0 + 4u * lane;
        const uint32_t ring0 = smem_u32(ring + ((size_t)team * p.D + (size_t)half * Dw) * p.slot_bytes);
        const uint32_t bar0 = smem_u32(&bars[team * p.D + half * Dw]);
        volatile int *team_flag = reinterpret_cast<volatile int *>(smem + lay.flag) + team;
        const int stream_threads = teams * stride * 32;
        auto team_sync = [&]() {                                      // the warp alone, or the two warps of the team
            if (pp) asm volatile("bar.sync %0, 64;" ::"r"(2 + team) : "memory");
            else __syncwarp();
        };
        bool zeroed = false;
        const uint32_t lt_mask = (1u << lane) - 1u;
        const uint32_t items0 = smem_u32(items);
        uint32_t issued = 0, consumed = 0;                            // copies asked for / used up by this team
        uint32_t slot = 0, parity = 0, islot = 0;                     // of this warp's Dw slots: consumed % Dw, its phase, issued % Dw
        StepBuf b0, b1;                                               // pipeline registers, live across items
        const uint32_t zeros = smem_u32(zero_group);
        float racc[kRegRows > 0 ? kRegRows : 1];                      // register-held sums of local rows 0 .. kRegRows-1
#pragma unroll
        for (int i = 0; i < (kRegRows > 0 ? kRegRows : 1); ++i) racc[i] = 0.f;
        const uint32_t reg_lim = cell0 + (uint32_t)min(kRegRows, p.R) * 128u;

        for (int rb = r_begin;; rb += p.cap) {                        // at least one trip: the teams meet at a barrier in it
            const int cnt = failed ? 0 : max(0, min(p.cap, r_end - rb));
            // ---- column of rank r: the block of keep words that holds it, then the word, then the bit
#pragma unroll 1
            for (int i = half * 32 + lane; i < cnt; i += 32 * stride) {
                const int r = rb + i;
                int j;
                uint16_t xb;
                if (from_list) {
                    j = min(max(__ldcg(p.list_idx + r), 0), p.K - 1);
                    xb = __ldcg(p.list_val + r);
                } else {
                // the block of 32 keep words that holds rank r (the last one with blk[e] <= r), the word in it
                // (the last one with wrel[w] <= what is left) ...
                // (both tables are nondecreasing, so "the last entry <= r" is a count of such entries, and counting
                // takes independent loads where a binary search takes dependent ones: up to eight blocks in one
                // round, the 32 words of a block in two -- quarters, then the eight words of the quarter)
                int e = 0;
                if (nblk <= 8) {
#pragma unroll
                    for (int u = 1; u < 8; ++u) e += (u < nblk && myblk[u] <= r) ? 1 : 0;
                } else {
#pragma unroll 1
                    for (int step = 1 << (31 - __clz(nblk - 1)); step; step >>= 1)
                        if (e + step < nblk && myblk[e + step] <= r) e += step;
                }
                int k = r - myblk[e], w = 32 * e;
                {
                    int quarter = 0;
#pragma unroll
                    for (int u = 8; u < 32; u += 8) quarter += (w + u < nwords && wrel[w + u] <= k) ? 1 : 0;
                    w += 8 * quarter;
                    int in_quarter = 0;
#pragma unroll
                    for (int u = 1; u < 8; ++u) in_quarter += (w + u < nwords && wrel[w + u] <= k) ? 1 : 0;
                    w += in_quarter;
                }
                k -= wrel[w];
                // ... and the bit in it: halve the word, keep the half that holds the wanted set bit
                const uint32_t word = kbw[w];
                int pos = 0;
#pragma unroll
                for (int sh = 16; sh; sh >>= 1) {
                    const int c = __popc((word >> pos) & ((1u << sh) - 1u));
                    if (k >= c) { k -= c; pos += sh; }
                }
                j = 32 * w + pos;
                if (kExtras && p.swiglu_in) xb = (uint16_t)swiglu_half_bits(__ldg(p.swiglu_in + j), __ldg(p.swiglu_in + p.K + j));
                else xb = __ldg(p.x + j);                            // x went through L1 in the thresholding pass
                }
                items[i] = make_int2(j, (int)xb);
                if (!from_list && part == 0 && sl == 0) {
                    p.idx[r] = j;
                    p.val[r] = xb;
                }
                if (s < p.S) {
                    // the two offsets of sub-block (j, s): from the block's window of the table if they are in it
                    const int wq = j * p.S + s - win_w0;
                    uint32_t o0, o1;
                    if (__builtin_expect(wq >= 0 && wq + 1 < win_n, 1)) {
                        o0 = win[wq];
                        o1 = win[wq + 1];
                    } else {
                        o0 = p.meta[(size_t)j * p.S + s];
                        o1 = p.meta[(size_t)j * p.S + s + 1];
                    }
                    imeta[i] = make_uint2(o0, (o1 - o0) * 16u);
                }
            }
            // The accumulators take the place of the window: every team has to be through with its look-ups
            // before any team clears its slab.  (Teams with more than `cap` columns come back here for their
            // later batches, and find the offsets in global memory then.)
            if (rb == r_begin) asm volatile("bar.sync 1, %0;" ::"r"(stream_threads) : "memory");
            else team_sync();
            win_n = 0;
            if (rb + p.cap >= r_end && (cnt == 0 || s >= p.S)) break;
            if (cnt == 0 || s >= p.S) continue;
            // ---- a2: keep D copies in flight.  The team issues the first D of a batch and refills a slot whenever
            // it has finished with it.  Every lane calls issue(), converged, and keeps the ring position; one
            // elected lane (elect.sync) runs the two instructions under a predicate -- 3 % faster at 28672 x 8192
            // than a branch on lane 0, around which the warp diverges and reconverges for every sub-block.
            auto issue_im = [&](const uint2 im) {
                bulk_load_elected(ring0 + islot * (uint32_t)p.slot_bytes, p.stream + (size_t)im.x * 16, im.y,
                                  bar0 + 8u * islot);
                ++issued;
                if (++islot == (uint32_t)Dw) islot = 0;
            };
#pragma unroll 1
            for (int k = 0, i = half; k < Dw && i < cnt; ++k, i += stride) issue_im(imeta[i]);
            if (!zeroed) {                                          // clear the slab while the first copies fly
                float4 *slab4 = reinterpret_cast<float4 *>(acc + (size_t)team * slab_words);
#pragma unroll 1
                for (int i = half * 32 + lane; i < slab_words / 4; i += 32 * stride) slab4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                zeroed = true;
                team_sync();
            }
            for (int i = half; i < cnt; i += stride) {
                uint32_t xbits;                                       // the column's activation: asked for before the wait
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(xbits) : "r"(items0 + 8u * (uint32_t)i + 4u));
                if (!failed && !mbar_wait_bounded(bar0 + 8u * slot, parity, p.spin_limit)) failed = true;
                failed = __any_sync(kFull, failed);
                if (__builtin_expect(failed, 0)) {
                    // The copies still in flight are awaited below.  A warp that gave up keeps meeting its partner at
                    // the hand-overs of this batch, so that nobody waits for it in vain.
                    if (!pp) break;
                    if (lane == 0) *team_flag = 1;
                    if (i > 0) team_sync();
                    if (i + 1 < cnt) team_sync();
                    continue;
                }
                const uint32_t sub = ring0 + slot * (uint32_t)p.slot_bytes;
                // what the refill at the end of this sub-block will need, read now so that it does not wait then
                const bool refill = i + stride * Dw < cnt;
                const uint2 next_im = refill ? imeta[i + stride * Dw] : make_uint2(0u, 0u);
                const uint16_t xj = (uint16_t)xbits;
                // ---- a3 + a4.  Header: groups per lane, vectors and steps (see kSubHeader).
                uint32_t gl, hw;
                asm volatile("ld.shared.u8 %0, [%1];" : "=r"(gl) : "r"(sub + lane));
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(hw) : "r"(sub + 32));       // vectors | steps << 16
                const uint32_t steps = hw >> 16, Gs = hw & 0xFFFFu;
                const uint32_t vbase = sub + kSubHeader, rbase = vbase + 16 * Gs;
                uint32_t cum = 0, cell = cell0;
                const uint32_t spare = cell0 + (uint32_t)p.R * 128u;
                step_fetch(b0, gl, 0, steps, cum, lt_mask, vbase, rbase, zeros);
                step_fetch(b1, gl, 1, steps, cum, lt_mask, vbase, rbase, zeros);
                // nothing above touches the accumulator: here the partner hands it over (it has finished the
                // column before this one)
                if (pp && i > 0) team_sync();
                step_decode<kRegRows>(b0, cell, spare, reg_lim);                                    // step 0
                step_fetch(b0, gl, 2, steps, cum, lt_mask, vbase, rbase, zeros);
                uint32_t q = 1;
#pragma unroll 2
                for (; q + 1 < steps; q += 2) {                                            // two real steps per pass
                    step_decode<kRegRows>(b1, cell, spare, reg_lim);                                // step q
                    step_finish(b0, xj);                                                   // step q-1
                    step_fetch(b1, gl, q + 2, steps, cum, lt_mask, vbase, rbase, zeros);
                    step_decode<kRegRows>(b0, cell, spare, reg_lim);                                // step q+1
                    step_finish(b1, xj);                                                   // step q
                    step_fetch(b0, gl, q + 3, steps, cum, lt_mask, vbase, rbase, zeros);
                }
                if (q < steps) {                                                           // one real step left
                    step_decode<kRegRows>(b1, cell, spare, reg_lim);
                    step_finish(b0, xj);
                    step_finish(b1, xj);
                } else {                                                                   // only the last one to finish
                    step_finish(b0, xj);
                }
                if (kRegRows > 0) {
                    // collect this column's products of the register rows and leave their cells empty for the next
#pragma unroll
                    for (int i = 0; i < kRegRows; ++i)
                        if (i < p.R) {
                            racc[i] += lds_f32(cell0 + (uint32_t)i * 128u);
                            sts_f32(cell0 + (uint32_t)i * 128u, 0.f);
                        }
                }
                // The slot's contents were consumed by loads whose values have been used, and the barrier orders
                // every lane's reads before this point: the copy may overwrite it.
                __syncwarp();
                if (refill) issue_im(next_im);
                if (pp && i + 1 < cnt) team_sync();                 // the accumulator goes to the partner
                ++consumed;
                if (++slot == (uint32_t)Dw) { slot = 0; parity ^= 1u; }
            }
            team_sync();                                          // items / imeta are rewritten by the next batch
            if (pp && *team_flag) failed = true;                // both warps of a team stop together
            if (failed || rb + p.cap >= r_end) break;
        }
        if (kRegRows > 0 && zeroed) {                                 // the register rows go to the slab for the merge
#pragma unroll
            for (int i = 0; i < kRegRows; ++i)
                if (i < p.R) sts_f32(cell0 + (uint32_t)i * 128u, racc[i]);
        }
        if (__builtin_expect(!zeroed && s < p.S, 0)) {                // a team without columns still owns a slab
            float4 *slab4 = reinterpret_cast<float4 *>(acc + (size_t)team * slab_words);
#pragma unroll 1
            for (int i = lane; i < slab_words / 4; i += 32) slab4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (__builtin_expect(failed, 0)) {
            // give the copies that are still in flight a last (bounded) chance to land before the block goes on
#pragma unroll 1
            for (; consumed < issued; ++consumed) {
                mbar_wait_bounded(bar0 + 8u * slot, parity, p.spin_limit);
                if (++slot == (uint32_t)Dw) { slot = 0; parity ^= 1u; }
            }
            if (lane == 0) atomicOr(p.status, kStatusTimeout);
        }
    }
    __syncthreads();

    if (merge == 1) {
        // ---- a5 by bulk reduce-add.  The block adds its G accumulators; the row segments of its slabs (32*C rows
        // of y each, see the row map) are then dealt to the blocks of the cluster, a block adds its peers' sums
        // for its segments (through distributed shared memory), and the copy engine adds the result into y
        // (cp.reduce.async.bulk, FP32 add at L2).  y was cleared by all blocks at the start; the ticket makes
        // sure of it.
        if (warp == nwarps - 1 && lane == 0) {                      // every block's share of y is cleared by now
            const bool low_half = y_ticket < gridDim.x;
            bool ok = false;
            for (uint32_t it = 0; it < p.spin_limit; ++it) {
                const uint32_t cur = ld_relaxed_u32(&p.tickets[0]);
                if (low_half ? (cur >= gridDim.x) : (cur < gridDim.x)) { ok = true; break; }
                __nanosleep(64);
            }
            __threadfence();
            // the clearing stores of the other blocks (generic proxy) come before this block's reduce-adds
            // (asynchronous proxy) to the same addresses
            asm volatile("fence.proxy.async.global;" ::: "memory");
            if (__builtin_expect(!ok, 0)) atomicOr(p.status, kStatusTimeout);
        }
        __syncwarp();
        // add the G accumulators of every slab into the first one
        const int group_words = Sc * slab_words;
        if (G > 1) {
            float4 *acc4 = reinterpret_cast<float4 *>(acc);
            const int group4 = group_words / 4;
#pragma unroll 1
            for (int q4 = tid; q4 < group4; q4 += nthreads) {
                float4 v = acc4[q4];
#pragma unroll 2
                for (int gg = 1; gg < G; ++gg) {
                    const float4 t = acc4[(size_t)gg * group4 + q4];
                    v.x += t.x; v.y += t.y; v.z += t.z; v.w += t.w;
                }
                acc4[q4] = v;
            }
        }
        const int seg = p.S == 1 ? 16 : p.C, nseg = idiv_small(p.R + seg - 1, seg), seg4 = seg * 8;
        const int owned = (Sc * nseg - crank + cl - 1) / cl;   // segments crank, crank + cl, ...
        if (cl > 1) {
            cluster_sync();                                         // the peers' sums are complete
            for (int t = tid; t < owned * seg4; t += nthreads) {
                const int sg = crank + cl * (t / seg4), q4 = t % seg4;
                const int fsl = sg / nseg, i0 = (sg - fsl * nseg) * seg;
                if (i0 * 32 + q4 * 4 >= p.R * 32) continue;         // a slab's last segment may be short
                float4 *cellp = reinterpret_cast<float4 *>(acc + (size_t)fsl * slab_words + (size_t)i0 * 32 + (size_t)q4 * 4);
                float4 v = *cellp;
                for (int b = 1; b < cl; ++b) {
                    const float4 u = ld_cluster_f4(smem_u32(cellp), (uint32_t)((crank + b) % cl));
                    v.x += u.x; v.y += u.y; v.z += u.z; v.w += u.w;
                }
                // no other block reads this place: a block reads only the segments it owns, from everybody
                *cellp = v;
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        // The row map makes local rows [kC, kC + C) of a slab 32*C consecutive rows of y, in accumulator
        // order (with one slab the whole accumulator is y itself): each such segment is one bulk reduce-add.
        {
#pragma unroll 1
            for (int o = tid; o < owned; o += nthreads) {
                const int sg = crank + cl * o;
                const int fsl = idiv_small(sg, nseg), k = sg - fsl * nseg, sfull = part * Sc + fsl;
                if (sfull >= p.S) continue;
                const int i0 = k * seg, i1 = min(p.R, i0 + seg);
                // tile_row(S, C, sfull, 0, i0) for a segment's first local row i0 = k * seg, without its divisions:
                // seg is C (one chunk of the row map) unless there is one slab, whose rows are y in order
                const int64_t row0 = p.S == 1 ? (int64_t)i0 * 32 : ((int64_t)(k * p.S + sfull) * p.C) * 32;
                if (row0 >= p.M) continue;
                const int nrows = min((i1 - i0) * 32, p.M - (int)row0);
                const uint32_t bytes = ((uint32_t)nrows * 4u) & ~15u;
                const float *src = acc + (size_t)fsl * slab_words + (size_t)i0 * 32;
                if (bytes)
                    asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;" ::"l"(p.y + row0),
                                 "r"(smem_u32(src)), "r"(bytes)
                                 : "memory");
#pragma unroll 1
                for (int i = (int)(bytes >> 2); i < nrows; ++i)
                    if (src[i] != 0.f) atomicAdd(p.y + row0 + i, src[i]);
            }
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // shared memory may go once it has been read
        }
        if (cl > 1) cluster_sync();                               // no block leaves while a peer may still read it
        if (!kExtras || p.ep_kind == 0) return;
        fused_epilogue(EpilogueArgs{p.y, p.tickets, p.status, p.spin_limit, p.M, p.ep_kind, p.ep_out, p.ep_tau, p.ep_idx,
                                    p.ep_val, p.ep_count});
        return;
    }
    {
        // ---- a5, ordered (clusters are not used with this merge).  Stage 1: add the G accumulators, store the block's partial (accumulator layout, no slack rows)
        const int tile_words = p.R * 32, part_words = p.Sc * tile_words;
        {
            float4 *mine4 = reinterpret_cast<float4 *>(p.partials + (size_t)blockIdx.x * part_words);
            const float4 *acc4 = reinterpret_cast<const float4 *>(acc);
            const int tile4 = tile_words >> 2, slab4 = slab_words >> 2, group4 = p.Sc * slab4;
            for (int fsl = 0; fsl < p.Sc; ++fsl)
                for (int q4 = tid; q4 < tile4; q4 += nthreads) {
                    const float4 *src = acc4 + fsl * slab4 + q4;
                    float4 v = src[0];
                    for (int gg = 1; gg < p.G; ++gg) {
                        const float4 t = src[gg * group4];
                        v.x += t.x; v.y += t.y; v.z += t.z; v.w += t.w;
                    }
                    __stcg(mine4 + fsl * tile4 + q4, v);
                }
        }
        __syncthreads();
        if (tid == 0) {
            __threadfence();                                          // the block's stores, ordered by the barrier above
            atomicAdd(&p.tickets[0], 1u);
            bool ok = false;
            for (uint32_t it = 0; it < p.spin_limit; ++it) {
                if (ld_acquire_u32(&p.tickets[0]) >= gridDim.x) { ok = true; break; }
                __nanosleep(32);
            }
            if (__builtin_expect(!ok, 0)) atomicOr(p.status, kStatusTimeout);
        }
        __syncthreads();

        // ---- a5, stage 2: the nK blocks of a part share its words; partial b of this part = block b*P + part.
        // The block's words are cut into chunks of 32; the warps split (chunk, range of partials) pairs so that
        // every lane has up to 16 loads in flight, then the ranges are added in a fixed order.
        {
            float *red = reinterpret_cast<float *>(smem + lay.acc);   // the accumulators are no longer needed
            const int wpc = (((part_words + nK - 1) / nK) + 31) & ~31;
            const int wb = kslice * wpc, we = min(part_words, wb + wpc);
            const int nchunks = max(0, (we - wb + 31) >> 5);
            const size_t stride = (size_t)p.P * part_words;
            for (int c0 = 0; c0 < nchunks; c0 += nwarps) {
                const int pass_chunks = min(nwarps, nchunks - c0);
                const int nsplit = nwarps / pass_chunks;              // warps per chunk in this pass
                const int my_chunk = warp % pass_chunks, my_split = warp / pass_chunks;
                const int word = wb + 32 * (c0 + my_chunk) + lane;
                if (my_split < nsplit) {
                    float sum = 0.f;
                    if (word < we) {
                        const int per = (nK + nsplit - 1) / nsplit;
                        const int b_lo = my_split * per, b_hi = min(nK, b_lo + per);
                        const float *src = p.partials + (size_t)part * part_words + word;
                        for (int b0 = b_lo; b0 < b_hi; b0 += 16) {
                            float t[16];
    #pragma unroll
                            for (int k = 0; k < 16; ++k)
                                t[k] = b0 + k < b_hi ? __ldcg(src + (size_t)(b0 + k) * stride) : 0.f;
    #pragma unroll
                            for (int k = 0; k < 16; ++k) sum += t[k];
                        }
                    }
                    red[(my_split * pass_chunks + my_chunk) * 32 + lane] = sum;
                }
                __syncthreads();
                if (warp < pass_chunks) {
                    const int w2 = wb + 32 * (c0 + warp) + lane;
                    if (w2 < we) {
                        float total = 0.f;
                        for (int sp = 0; sp < nsplit; ++sp) total += red[(sp * pass_chunks + warp) * 32 + lane];
                        const int fsl = w2 / tile_words, rem = w2 - fsl * tile_words;
                        const int sfull = part * p.Sc + fsl;
                        const int64_t row = tile_row(p.S, p.C, sfull, rem & 31, rem >> 5);
                        if (sfull < p.S && row < p.M) p.y[row] = total;
                    }
                }
                __syncthreads();
            }
        }
    }
    __syncthreads();
    if (tid == 0) {
        const uint32_t t = atomicAdd(&p.tickets[1], 1u);
        if (t == gridDim.x - 1) {                                  // last one out resets both tickets
            atomicExch(&p.tickets[0], 0u);
            atomicExch(&p.tickets[1], 0u);
        }
    }
}

struct FusedPlan {
    int G, Sc, P, D, cl, pp, mix, slot_bytes, cap, threads, grid, merge;
    size_t smem;
};

inline size_t fused_smem_bytes(int R, int K, int G, int Sc, int D, int slot_bytes, int cap)
{
    return fused_smem_layout(R, K, G * Sc, D, slot_bytes, cap).total;
}
