// Persistent dataflow kernel for RHT blocks larger than one shared-memory tile (k >= 15).
//
// Work is cut into tasks of one 2^13-coordinate tile each, run by CTAs of 128 threads:
//   A(wb, t)  pass A of tile t of worker-block wb: consecutive coordinates, stages of
//             stride 1 .. 2^12, result written to slot (wb mod R) of a ring in the workspace;
//   B(wb, p)  pass B of panel p: 2^(k-13) rows (2^13 apart) x 2^(26-k) columns read back from
//             the slot, stages 2^13 .. 2^(k-1), then the fused epilogue.
// A worker-block is (RHT block r, local worker i), wb = r * n_local + i.  Tasks are claimed
// from one queue in the order  A(0) .. A(L-1), [A(s), B(s-L)] for s = L .., B(..) : pass B
// follows its pass A by L worker-blocks, close enough for the ring (R slots of 2^k floats) to
// stay in L2, far enough that the tiles it needs are normally finished.  Dependencies only
// point backwards in the queue, and a task waits only before it starts, so a CTA that waits
// never waits for work that is not already claimed by a running CTA.  Every wait is bounded:
// on expiry the kernel sets THC_STATUS_WAIT_TIMEOUT, raises an abort flag that ends all CTAs,
// and returns.
//
// Each CTA is four compute warps and one control warp, a producer/consumer pair over two tile
// buffers.  The control warp claims the next task, starts what does not depend on anything
// (sign words, the TMA load of a pass-A gradient tile, L2 prefetch of tiles the compute warps
// fetch themselves), waits for the task's dependency, starts the TMA load of a pass-B panel
// (completion on an mbarrier) and hands the descriptor over through a full/empty named-barrier
// handshake; the compute warps wait for the data, run the rounds and report on a `done`
// mbarrier.  The control warp also signals completions to the other CTAs, so that the release
// fence is not on the compute warps' path; it does so at the next hand-shake or, while it
// waits for a dependency, as soon as the `done` mbarrier says so: a wait never holds back the
// signal of an earlier task, which may be the very thing waited for.  Tiles sit in shared
// memory in TMA's 128-byte swizzle: 16-byte chunk c at c ^ ((c >> 3) & 7).
//
// Modes: compress (fp32 or bf16 gradients in, packed indices out), the same with fused scales,
// exact range (pass A as compress, the epilogue only takes min / max), decompress (sums of 8,
// 16 or 32 bits in, fp32 out), aggregate + decompress (all workers' 4-bit indices in, pass A
// sums their table values in byte lanes before it transforms; the sums are written only on
// request) and error feedback (a worker's own packed indices in, x - RHT^-1(X) out).  The 2^20
// block has a compile-time geometry (KB = 7); 2^21 and 2^22 have one for 4-bit compress.
//
// Fused scales (kCompressF32Fused; Section 5.3 notes that the norm exchange can run beside the
// RHT).  Pass A does not need the clamp bound M, only the epilogue of pass B does.  So every
// pass-A task also sums the squares of its tile in fp64; the control warp stores the sum,
// counts finished tiles per RHT block, and the CTA that finishes the last of a block's
// n_local * T tiles computes M = t_p * max_i ||x_i|| / sqrt(B) from the stored sums in a fixed
// order, writes it to `scales` and releases the block's pass-B tasks.  The queue trails pass B
// behind pass A by n_local - 1 more worker-blocks so that this is normally done in time.
// In this mode a_done[0..15] count finished tiles of block r in entry r mod 16 and
// a_done[16..31] count finished blocks of that residue.
//
// Counters (in the context's device block, all zero between launches; the last CTA to leave
// clears them):  head, exited, abort, a_done[R], b_done[R].  a_done[s] counts finished A tiles
// of slot s over the whole launch (generation g of the slot is complete at (g+1)*T),
// b_done[s] finished B panels (slot may be overwritten by generation g once it reaches g*T).
#pragma once
#include <cuda.h>
#include "thc_device.cuh"

namespace thc {

constexpr int kPLog2 = 13;                  // coordinates per pipeline tile
constexpr int kPElems = 1 << kPLog2;
constexpr int kPChunks = kPElems / 4;
constexpr int kPThreads = 128;                // compute threads of a CTA
constexpr int kPCtaThreads = 160;             // plus one control warp that runs the queue
constexpr int kPSignWords = 512;            // sign words: two slots of 256 (pass A) or one of 512
constexpr int kMaxRing = 320;                // ring slots: blocks of 2^15 need up to 280 to cover the tasks in flight
constexpr int kBlockConstMax = 256;         // per-block constants cached in shared memory
constexpr uint32_t kMaxPolls = 1u << 21;

enum PipeMode { kCompressF32, kCompressBF16, kDecompress8, kDecompress16, kDecompress32,
                kCompressF32Fused,     // fp32 compress that also computes the block scales (below)
                kErrorFeedback,        // e_i = x_i - RHT^-1(X_i) from worker i's own packed indices
                kRangeF32,             // exact min / max of the rotated coordinates per RHT block
                kAggDecompress };      // decompress straight from the workers' packed indices (PS line + estimate line)

// Layout inside DeviceBlock::counters.  Every CTA hits `head` and `abort` for every task and
// the completion counters of the slots in use: each gets its own 128-byte line (head, exited,
// abort) or 32-byte sector (per-slot counters), so that polls of one do not queue behind
// atomics on another.
struct alignas(32) PaddedCounter { uint32_t v; uint32_t pad[7]; };
struct PipeCounters {
    uint32_t head;   uint32_t pad0[31];
    uint32_t exited; uint32_t pad1[31];
    uint32_t abort;  uint32_t pad2[31];
    PaddedCounter a_done[kMaxRing];
    PaddedCounter b_done[kMaxRing];
};
static_assert(sizeof(PipeCounters) <= sizeof(DeviceBlock::counters), "counters do not fit the device block");

struct PipeParams {
    uint64_t d;
    uint64_t d_pad;
    uint64_t wb_count;         // nblocks * n_local
    uint64_t total_tasks;
    float   *ring;             // R slots of 2^k floats
    const float *scales;
    DeviceBlock *dev;
    uint32_t k;
    uint32_t kb;               // k - 13: log2 rows of a pass-B tile
    uint32_t n_local;
    uint32_t lag;              // L
    uint32_t ring_slots;       // R
    uint32_t granularity;
    uint32_t divisor;
    uint32_t round;
    uint32_t worker_base;
    float    c_block;
    // fused scales only
    double  *tile_sq;          // wb_count * T sums of squares, one per pass-A tile
    float   *scales_out;       // = scales, written by the kernel
    float2  *fused_const;      // per block (kappa, offset) of the quantiser, written with M
    double   t_p;
    uint32_t exact_range;      // scales = nblocks minima then nblocks maxima (else M per block)
    uint32_t nblocks;
    uint32_t *range_keys;      // range mode: nblocks min keys then nblocks max keys
    uint32_t b_swz_mask;       // run-time geometry, pass-B tiles: chunk c sits at c ^ ((c >> 3) & mask)
    uint32_t agg_n;            // kAggDecompress: workers whose table values are summed
    uint32_t agg_acc_bits;     // ... and the width of the sums written on request (outp.p[1])
    uint32_t b_tma;            // ... and are fetched by TMA in this many boxes of 256 rows (k = 21: one;
                               // k = 22: two, 64-byte rows with the 64-byte swizzle); 3: k = 15 .. 19, one
                               // 3-D box; 0: by the compute warps
};

struct PtrArrayP { const void *p[THC_MAX_WORKERS]; };
struct MutPtrArrayP { void *p[THC_MAX_WORKERS]; };

struct TaskInfo {              // published by thread 0 for the whole CTA
    uint32_t idx;              // tile / panel index; 0xFFFFFFFF = no task
    uint32_t is_b;
    uint32_t wl;               // local worker
    uint32_t r;                // RHT block
    uint32_t slot;             // ring slot
    uint32_t gen;              // generation of the slot
    uint32_t tma;              // tile arrives by TMA on the slot's mbarrier
    uint32_t phase;            // ... with this phase parity
    float    bcx, bcy;         // block constants (fused scales: they do not exist at launch)
};

struct TmaMaps {               // tensor maps: one per worker gradient, one for the ring
    CUtensorMap in[THC_MAX_WORKERS];
    CUtensorMap ring;
};

// ------------------------------------------------------------------------ small helpers
__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ uint64_t make_evict_first_policy()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ void cp_async16_hint(void *smem_dst, const void *gsrc,
                                                uint32_t src_bytes, uint64_t policy)
{
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2, %3;"
                 :: "r"(dst), "l"(gsrc), "r"(src_bytes), "l"(policy) : "memory");
}

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc)
{
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst), "l"(gsrc) : "memory");
}

__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// Named barriers: 1,2 = task slot full; 3,4 = task slot consumed; 5 = compute warps only.
// bar.sync / bar.arrive are warp-aligned instructions: the __syncwarp() makes sure the warp
// has reconverged after any single-thread section before it.
__device__ __forceinline__ void bar_sync(int id, int count)
{
    __syncwarp();
    asm volatile("bar.sync %0, %1;" :: "r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_arrive(int id, int count)
{
    __syncwarp();
    asm volatile("bar.arrive %0, %1;" :: "r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void compute_barrier() { bar_sync(5, kPThreads); }

__device__ __forceinline__ uint32_t atom_release_add(uint32_t *p, uint32_t v)
{
    uint32_t old;
    asm volatile("atom.release.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}

__device__ __forceinline__ float ld_relaxed_f32(const float *p)
{
    float v;
    asm volatile("ld.relaxed.gpu.global.f32 %0, [%1];" : "=f"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void red_release_add(uint32_t *p, uint32_t v)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}

// ------------------------------------------------------------------ mbarrier / TMA
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(bar);
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(a), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(bar);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(a), "r"(bytes) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(bar);
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(a) : "memory");
}

// Non-blocking: has the phase with this parity completed?
__device__ __forceinline__ bool mbar_test(uint64_t *bar, uint32_t parity)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(bar);
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(a), "r"(parity) : "memory");
    return done != 0;
}

// Bounded wait for a phase of the mbarrier; false if it did not complete within about a
// second (2^31 SM cycles; a try_wait may itself suspend the thread for a while, so the bound
// is on time, not on attempts).
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(bar);
    long long t0 = 0;
    for (uint32_t it = 0; it < (1u << 22); ++it) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(a), "r"(parity) : "memory");
        if (done) return true;
        if ((it & 63u) == 63u) {
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > (1ll << 31)) return false;
        }
    }
    return false;
}

// One 2-D tile: box of the tensor map at element coordinates (x, y) -> shared memory.
__device__ __forceinline__ void tma_load_2d(void *smem_dst, const CUtensorMap *map, int x, int y,
                                            uint64_t *bar, uint64_t policy)
{
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    const uint32_t b = (uint32_t)__cvta_generic_to_shared(bar);
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
                 ".L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
                 :: "r"(d), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(b), "l"(policy)
                 : "memory");
}

// One 3-D tile: box of the tensor map at element coordinates (x, y, z) -> shared memory.
__device__ __forceinline__ void tma_load_3d(void *smem_dst, const CUtensorMap *map, int x, int y, int z,
                                            uint64_t *bar, uint64_t policy)
{
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    const uint32_t b = (uint32_t)__cvta_generic_to_shared(bar);
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
                 ".L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;"
                 :: "r"(d), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(b), "l"(policy)
                 : "memory");
}

// Orders this thread's earlier generic-proxy accesses to shared memory before later
// async-proxy (TMA) writes to it.
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// The same for global memory: generic-proxy writes (made visible by an acquire) before this
// thread's later TMA reads of them.
__device__ __forceinline__ void fence_proxy_async_global()
{
    asm volatile("fence.proxy.async.global;" ::: "memory");
}

__device__ __forceinline__ void prefetch_l2(const void *p)
{
    asm volatile("prefetch.global.L2 [%0];" :: "l"(p));
}

__device__ __forceinline__ uint64_t make_evict_normal_policy()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ int pswz(int c) { return c ^ ((c >> 3) & 7); }

// Lane <-> unit permutation (swap bits 2 and 3): makes pairs of adjacent chunks per lane
// conflict-free in the XOR-swizzled tile.
__device__ __forceinline__ int swap_bits_2_3(int t)
{
    return (t & ~12) | ((t & 4) << 1) | ((t & 8) >> 1);
}

struct TaskId { uint32_t wb, idx, is_b, slot, gen; };

// Queue position -> task.  Order: A(0..L-1), then [A(s), B(s-L)] per worker-block, then the
// trailing B's.  T = tiles (= panels) per worker-block = 2^kb.
__device__ __forceinline__ TaskId decode_task(uint32_t q, const PipeParams &P)
{
    TaskId t;
    const uint32_t T = 1u << P.kb;
    const uint32_t wbc = (uint32_t)P.wb_count;
    const uint32_t head_tasks = P.lag << P.kb;
    const uint32_t mid_tasks = (wbc - P.lag) << (P.kb + 1);
    if (q < head_tasks) {
        t.wb = q >> P.kb; t.idx = q & (T - 1); t.is_b = 0;
    } else if (q - head_tasks < mid_tasks) {
        const uint32_t q1 = q - head_tasks;
        const uint32_t s = P.lag + (q1 >> (P.kb + 1));
        const uint32_t off = q1 & (2 * T - 1);
        t.is_b = off >= T;
        t.idx = off & (T - 1);
        t.wb = t.is_b ? s - P.lag : s;
    } else {
        const uint32_t q2 = q - head_tasks - mid_tasks;
        t.wb = wbc - P.lag + (q2 >> P.kb); t.idx = q2 & (T - 1); t.is_b = 1;
    }
    t.gen = t.wb / P.ring_slots;
    t.slot = t.wb - t.gen * P.ring_slots;
    return t;
}

template <bool COMPRESS>
__device__ __forceinline__ float2 block_constants(BlockRange b, uint32_t g, uint32_t divisor)
{
    return COMPRESS ? compress_constants(b) : decode_constants(b, g, divisor);
}

// ------------------------------------------------------------------ in-place tile rounds
// Butterfly stages on chunk-index bits [sp, sp+E) of a 2048-chunk tile (see fwht_round).
template <int E>
__device__ __forceinline__ void p_round(float4 *tile, int sp, int tid, int mask)
{
    constexpr int N = 1 << E;
    constexpr int kGroups = kPChunks >> E;
#pragma unroll 1
    for (int G = tid; G < kGroups; G += kPThreads) {
        const int low = G & ((1 << sp) - 1);
        const int base = ((G >> sp) << (sp + E)) | low;
        float4 v[N];
#pragma unroll
        for (int m = 0; m < N; ++m) { const int c = base + (m << sp); v[m] = tile[c ^ ((c >> 3) & mask)]; }
#pragma unroll
        for (int t = 0; t < E; ++t) {
#pragma unroll
            for (int m = 0; m < N; ++m)
                if (!(m & (1 << t))) butterfly(v[m], v[m | (1 << t)]);
        }
#pragma unroll
        for (int m = 0; m < N; ++m) { const int c = base + (m << sp); tile[c ^ ((c >> 3) & mask)] = v[m]; }
    }
}

__device__ __forceinline__ void p_rounds(float4 *tile, int lo, int hi, int tid, int mask)
{
    int sp = lo;
    while (sp < hi) {
        const int e = min(4, hi - sp);
        switch (e) {
        case 4: p_round<4>(tile, sp, tid, mask); break;
        case 3: p_round<3>(tile, sp, tid, mask); break;
        case 2: p_round<2>(tile, sp, tid, mask); break;
        default: p_round<1>(tile, sp, tid, mask); break;
        }
        sp += e;
        compute_barrier();
    }
}

// ------------------------------------------------------------------------------- pass A
// A tile is 256 rows of 8 chunks (32 coordinates); row r, chunk cc sits at r*8 + (cc ^ (r&7)).
//
// First round, in place: sign flip (compress), stages of stride 1 and 2 inside each chunk,
// then stride 4, 8, 16 across the eight chunks of a row.  Thread (warp w, lane l) owns rows
// 64 w + l and 64 w + 32 + l: a warp works on the same 64 rows here and in the next round
// (round_rows_0_3), so only a warp barrier separates the two.
// With SQ the thread's sum of squares of the 64 inputs (fp64, four interleaved partial
// sums combined in a fixed order) is returned.
template <bool FLIP, bool SQ>
__device__ __forceinline__ double pass_a_round1(float4 *tile, const uint32_t *sw, int tid)
{
    const int x = tid & 7;
    const int r0 = ((tid >> 5) << 6) | (tid & 31);
    double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
    // The two rows are independent: a loop of two iterations instead of 16 chunks at once
    // halves the code of this round (the kernel is large enough for instruction fetch to show).
#pragma unroll 1
    for (int g = 0; g < 2; ++g) {
        float4 v[8];
        float4 *row = tile + (r0 + 32 * g) * 8;
#pragma unroll
        for (int m = 0; m < 8; ++m) v[m] = row[m ^ x];
        if (SQ) {
#pragma unroll
            for (int m = 0; m < 8; ++m) {
                a0 = fma((double)v[m].x, (double)v[m].x, a0);
                a1 = fma((double)v[m].y, (double)v[m].y, a1);
                a2 = fma((double)v[m].z, (double)v[m].z, a2);
                a3 = fma((double)v[m].w, (double)v[m].w, a3);
            }
        }
        if (FLIP) {
            const uint32_t w = sw[r0 + 32 * g];
#pragma unroll
            for (int m = 0; m < 8; ++m) v[m] = flip4(v[m], w >> (m * 4));
        }
#pragma unroll
        for (int m = 0; m < 8; ++m) v[m] = stages01(v[m]);
#pragma unroll
        for (int t = 0; t < 3; ++t) {
#pragma unroll
            for (int m = 0; m < 8; ++m)
                if (!(m & (1 << t))) butterfly(v[m], v[m | (1 << t)]);
        }
#pragma unroll
        for (int m = 0; m < 8; ++m) row[m ^ x] = v[m];
    }
    return SQ ? (a0 + a1) + (a2 + a3) : 0.0;
}

// First round of a pass-A tile of a bf16 gradient that lies wholly inside the vector: the TMA
// unit has put the 16 KB of bf16 (256 rows of 64 bytes, 64-byte swizzle) into the upper half of
// the tile buffer.  Every thread reads its two rows into registers; after a block barrier
// (the fp32 rows written next overlap other threads' bf16 rows) the values are widened to fp32
// (exact) and the round goes on as pass_a_round1 does.
__device__ __forceinline__ void pass_a_round1_bf16(float4 *tile, const uint32_t *sw, int tid)
{
    const int x = tid & 7;
    const int r0 = ((tid >> 5) << 6) | (tid & 31);
    const uint4 *stage = reinterpret_cast<const uint4 *>(tile) + kPChunks / 2;
    uint4 raw[8];
#pragma unroll
    for (int g = 0; g < 2; ++g) {
        const int row = r0 + 32 * g;
#pragma unroll
        for (int q = 0; q < 4; ++q) raw[4 * g + q] = stage[row * 4 + (q ^ ((row >> 1) & 3))];
    }
    compute_barrier();
    // one row per iteration (see pass_a_round1); the second row's staged words move down
#pragma unroll 1
    for (int g = 0; g < 2; ++g) {
        float4 v[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint4 t4 = raw[i];
            v[2 * i] = make_float4(__uint_as_float(t4.x << 16), __uint_as_float(t4.x & 0xFFFF0000u),
                                   __uint_as_float(t4.y << 16), __uint_as_float(t4.y & 0xFFFF0000u));
            v[2 * i + 1] = make_float4(__uint_as_float(t4.z << 16), __uint_as_float(t4.z & 0xFFFF0000u),
                                       __uint_as_float(t4.w << 16), __uint_as_float(t4.w & 0xFFFF0000u));
        }
        const uint32_t w = sw[r0 + 32 * g];
#pragma unroll
        for (int m = 0; m < 8; ++m) v[m] = flip4(v[m], w >> (m * 4));
#pragma unroll
        for (int m = 0; m < 8; ++m) v[m] = stages01(v[m]);
#pragma unroll
        for (int t = 0; t < 3; ++t) {
#pragma unroll
            for (int m = 0; m < 8; ++m)
                if (!(m & (1 << t))) butterfly(v[m], v[m | (1 << t)]);
        }
        float4 *row = tile + (r0 + 32 * g) * 8;
#pragma unroll
        for (int m = 0; m < 8; ++m) row[m ^ x] = v[m];
#pragma unroll
        for (int i = 0; i < 4; ++i) raw[i] = raw[i + 4];
    }
}

// First round of a pass-A tile of the inverse transform (decompress, error feedback): the same
// stages as pass_a_round1, but the thread fetches its two rows straight from global memory
// (the control warp has pulled the lines into L2) and de-quantises them in registers:
// sums Y -> m + Y (M - m)/(g n), or own indices z -> m + T[z] (M - m)/g  (Algorithm 2).
// A row of 32 coordinates is IN_BITS 32-bit words; a warp's rows are contiguous in memory.
template <int MODE, int BITS, int FREP>
__device__ __forceinline__ void pass_a_round1_inverse(float4 *tile, const unsigned char *src, float2 bc,
                                                      const float *ft, int tid)
{
    constexpr int IN_BITS = MODE == kDecompress8 ? 8 : MODE == kDecompress16 ? 16
                            : MODE == kDecompress32 ? 32 : BITS;
    const int x = tid & 7;
    const int r0 = ((tid >> 5) << 6) | (tid & 31);
    // the words of both rows first (all loads in flight together), then one row per iteration
    // (see pass_a_round1) with the second row's words moving down
    uint32_t w[2 * IN_BITS];
#pragma unroll
    for (int g = 0; g < 2; ++g) {
        const unsigned char *p = src + (size_t)(r0 + 32 * g) * (IN_BITS * 4);
        uint32_t *wg = w + g * IN_BITS;
        if constexpr (IN_BITS >= 4) {
#pragma unroll
            for (int q = 0; q < IN_BITS / 4; ++q) {
                const uint4 t4 = __ldg(reinterpret_cast<const uint4 *>(p) + q);
                wg[4 * q] = t4.x; wg[4 * q + 1] = t4.y; wg[4 * q + 2] = t4.z; wg[4 * q + 3] = t4.w;
            }
        } else if constexpr (IN_BITS == 3) {
            wg[0] = __ldg(reinterpret_cast<const uint32_t *>(p));
            wg[1] = __ldg(reinterpret_cast<const uint32_t *>(p) + 1);
            wg[2] = __ldg(reinterpret_cast<const uint32_t *>(p) + 2);
        } else if constexpr (IN_BITS == 2) {
            const uint2 t2 = __ldg(reinterpret_cast<const uint2 *>(p));
            wg[0] = t2.x; wg[1] = t2.y;
        } else {
            wg[0] = __ldg(reinterpret_cast<const uint32_t *>(p));
        }
    }
#pragma unroll 1
    for (int g = 0; g < 2; ++g) {
        float4 v[8];
#pragma unroll
        for (int m = 0; m < 8; ++m) {
            float sv[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int bit = (m * 4 + e) * IN_BITS;
                const uint32_t nxt = w[((bit >> 5) + 1) < IN_BITS ? (bit >> 5) + 1 : (bit >> 5)];
                const uint32_t val = IN_BITS == 32 ? w[bit >> 5]
                                     : __funnelshift_r(w[bit >> 5], nxt, bit & 31) & ((1u << (IN_BITS & 31)) - 1u);
                float yf;
                if (MODE == kErrorFeedback) yf = ft[val * FREP];
                else if (MODE == kDecompress32) yf = (float)val;
                else yf = __uint_as_float(0x4B000000u | val) - 8388608.0f;
                sv[e] = fmaf(yf, bc.x, bc.y);
            }
            v[m] = make_float4(sv[0], sv[1], sv[2], sv[3]);
        }
#pragma unroll
        for (int m = 0; m < 8; ++m) v[m] = stages01(v[m]);
#pragma unroll
        for (int t = 0; t < 3; ++t) {
#pragma unroll
            for (int m = 0; m < 8; ++m)
                if (!(m & (1 << t))) butterfly(v[m], v[m | (1 << t)]);
        }
        float4 *row = tile + (r0 + 32 * g) * 8;
#pragma unroll
        for (int m = 0; m < 8; ++m) row[m ^ x] = v[m];
#pragma unroll
        for (int q = 0; q < IN_BITS; ++q) w[q] = w[q + IN_BITS];
    }
}

// First round of a pass-A tile of thc_aggregate_decompress: the PS line and the estimate line of
// Algorithm 2 in one place.  The thread fetches the packed indices of its two rows from every
// worker, adds up the table values (in byte lanes, then exactly in floats: the sums stay below
// 2^24 and equal the integer sums thc_aggregate writes), optionally writes the sums, and goes on
// as pass_a_round1_inverse does with v = m + Y (M - m)/(g n).  4-bit indices and table values
// below 128 only (the host sends every other configuration through the two separate kernels).
__device__ __forceinline__ void pass_a_round1_aggregate(float4 *tile, const PtrArrayP &in, uint32_t agg_n,
                                                        size_t byte_off, float2 bc,
                                                        void *sum_out, size_t coord_off, uint32_t acc_bits, int tid,
                                                        const uint32_t (&tb)[4], uint32_t swar_chunk)
{
    const int x = tid & 7;
    const int r0 = ((tid >> 5) << 6) | (tid & 31);
    float4 v[16];
#pragma unroll
    for (int m = 0; m < 16; ++m) v[m] = make_float4(0.f, 0.f, 0.f, 0.f);
    {
        // 4-bit indices, table values below 128: four look-ups per byte-permute instruction and
        // sums in byte lanes (see aggregate_b4w8_kernel), `swar_chunk` workers at a time so that
        // no byte overflows; the byte sums are then widened exactly into the float accumulators.
#pragma unroll 1
        for (uint32_t i0 = 0; i0 < agg_n; i0 += swar_chunk) {
            uint32_t acc[2][8];
#pragma unroll
            for (int g = 0; g < 2; ++g)
#pragma unroll
                for (int q = 0; q < 8; ++q) acc[g][q] = 0u;
            const uint32_t i1 = min(agg_n, i0 + swar_chunk);
#pragma unroll 2
            for (uint32_t i = i0; i < i1; ++i) {
                const unsigned char *src = static_cast<const unsigned char *>(in.p[i]) + byte_off;
#pragma unroll
                for (int g = 0; g < 2; ++g) {
                    const uint4 t4 = __ldg(reinterpret_cast<const uint4 *>(src + (size_t)(r0 + 32 * g) * 16));
                    const uint32_t words[4] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const uint32_t a = words[h], b = a ^ 0x88888888u;
                        uint32_t lo, hi, lo2, hi2;
                        asm("prmt.b32 %0, %1, %2, %3;" : "=r"(lo) : "r"(tb[0]), "r"(tb[1]), "r"(a));
                        asm("prmt.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(tb[2]), "r"(tb[3]), "r"(b));
                        asm("prmt.b32 %0, %1, %2, %3;" : "=r"(lo2) : "r"(tb[0]), "r"(tb[1]), "r"(a >> 16));
                        asm("prmt.b32 %0, %1, %2, %3;" : "=r"(hi2) : "r"(tb[2]), "r"(tb[3]), "r"(b >> 16));
                        acc[g][2 * h] += lo + hi;
                        acc[g][2 * h + 1] += lo2 + hi2;
                    }
                }
            }
#pragma unroll
            for (int g = 0; g < 2; ++g)
#pragma unroll
                for (int m = 0; m < 8; ++m) {
                    const uint32_t wv = acc[g][m];
                    v[8 * g + m].x += __uint_as_float(__byte_perm(wv, 0x4B000000u, 0x7440)) - 8388608.0f;
                    v[8 * g + m].y += __uint_as_float(__byte_perm(wv, 0x4B000000u, 0x7441)) - 8388608.0f;
                    v[8 * g + m].z += __uint_as_float(__byte_perm(wv, 0x4B000000u, 0x7442)) - 8388608.0f;
                    v[8 * g + m].w += __uint_as_float(__byte_perm(wv, 0x4B000000u, 0x7443)) - 8388608.0f;
                }
        }
    }
    if (sum_out != nullptr) {
        // the sums of the thread's two rows of 32 coordinates, acc_bits each
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            const size_t j = coord_off + (size_t)(r0 + 32 * g) * 32;
            uint32_t y[32];
#pragma unroll
            for (int m = 0; m < 8; ++m) {
                y[4 * m] = (uint32_t)v[8 * g + m].x; y[4 * m + 1] = (uint32_t)v[8 * g + m].y;
                y[4 * m + 2] = (uint32_t)v[8 * g + m].z; y[4 * m + 3] = (uint32_t)v[8 * g + m].w;
            }
            if (acc_bits == 8) {
                uint4 *o = reinterpret_cast<uint4 *>(static_cast<unsigned char *>(sum_out) + j);
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    uint32_t ww[4];
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int b0 = 16 * q + 4 * c;
                        ww[c] = y[b0] | (y[b0 + 1] << 8) | (y[b0 + 2] << 16) | (y[b0 + 3] << 24);
                    }
                    o[q] = make_uint4(ww[0], ww[1], ww[2], ww[3]);
                }
            } else if (acc_bits == 16) {
                uint4 *o = reinterpret_cast<uint4 *>(static_cast<unsigned char *>(sum_out) + 2 * j);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t ww[4];
#pragma unroll
                    for (int c = 0; c < 4; ++c) ww[c] = y[8 * q + 2 * c] | (y[8 * q + 2 * c + 1] << 16);
                    o[q] = make_uint4(ww[0], ww[1], ww[2], ww[3]);
                }
            } else {
                uint4 *o = reinterpret_cast<uint4 *>(static_cast<unsigned char *>(sum_out) + 4 * j);
#pragma unroll
                for (int q = 0; q < 8; ++q) o[q] = make_uint4(y[4 * q], y[4 * q + 1], y[4 * q + 2], y[4 * q + 3]);
            }
        }
    }
#pragma unroll
    for (int m = 0; m < 16; ++m) {
        v[m].x = fmaf(v[m].x, bc.x, bc.y); v[m].y = fmaf(v[m].y, bc.x, bc.y);
        v[m].z = fmaf(v[m].z, bc.x, bc.y); v[m].w = fmaf(v[m].w, bc.x, bc.y);
    }
#pragma unroll
    for (int m = 0; m < 16; ++m) v[m] = stages01(v[m]);
#pragma unroll
    for (int t = 0; t < 3; ++t) {
#pragma unroll
        for (int m = 0; m < 16; ++m)
            if (!(m & (1 << t))) butterfly(v[m], v[m | (1 << t)]);
    }
#pragma unroll
    for (int g = 0; g < 2; ++g) {
        float4 *row = tile + (r0 + 32 * g) * 8;
#pragma unroll
        for (int m = 0; m < 8; ++m) row[m ^ x] = v[8 * g + m];
    }
}

// Round on row bits 0..3: thread (rg = tid >> 3, cc = tid & 7) owns chunk cc of rows
// 16 rg + m.  Serves pass A (second round) and the first round of a k = 20 pass-B tile, whose
// two 128-row halves are simply rows 0..255.
__device__ __forceinline__ void round_rows_0_3(float4 *tile, int tid)
{
    float4 *mine = tile + ((tid >> 3) << 7);
    const int cc = tid & 7;
    float4 *q[8];
#pragma unroll
    for (int x = 0; x < 8; ++x) q[x] = mine + (cc ^ x);
    float4 v[16];
#pragma unroll
    for (int m = 0; m < 16; ++m) v[m] = q[m & 7][8 * m];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
#pragma unroll
        for (int m = 0; m < 16; ++m)
            if (!(m & (1 << t))) butterfly(v[m], v[m | (1 << t)]);
    }
#pragma unroll
    for (int m = 0; m < 16; ++m) q[m & 7][8 * m] = v[m];
}

// Last round of a pass-A tile (row bits 4..7): thread (rl = tid >> 3, cc = tid & 7) owns chunk
// cc of rows rl + 16 m; the result goes straight to the ring, 512 contiguous bytes per warp.
__device__ __forceinline__ void pass_a_round3_store(const float4 *tile, float *dst, int tid)
{
    const int rl = tid >> 3, cc = tid & 7;
    const float4 *mine = tile + rl * 8 + (cc ^ (rl & 7));
    float4 v[16];
#pragma unroll
    for (int m = 0; m < 16; ++m) v[m] = mine[m << 7];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
#pragma unroll
        for (int m = 0; m < 16; ++m)
            if (!(m & (1 << t))) butterfly(v[m], v[m | (1 << t)]);
    }
    float4 *out = reinterpret_cast<float4 *>(dst) + tid;
#pragma unroll
    for (int m = 0; m < 16; ++m) out[m << 7] = v[m];
}

// ------------------------------------------------------------------------------- pass B
struct EpilogueCtx {
    uint64_t j_tile;        // coordinate of (row 0, column 0) of the tile in the worker's vector
    float kappa, half_g, gf, c_block;
    uint32_t lut;           // this lane's address into the quantiser table (lut_lane_addr)
    uint32_t worker, round;
    unsigned char *packed;
    float *rotated;
    float *out;
    const float *xsub;      // error feedback: the output is xsub - (inverse transform)
    uint64_t d;
    const uint32_t *sw;
    int words_per_row;
};

// RANGE: the unit only feeds the running minimum / maximum (as ordered keys) of the rotated
// coordinates (Algorithm 1's preliminary stage).
template <bool COMPRESS, int BITS, bool IDENTITY, bool RANGE = false>
__device__ __forceinline__ void epilogue_unit(const float4 &va, const float4 &vb, uint64_t j, int row,
                                              int uu, const EpilogueCtx &ep, const PhiloxKeys &keys,
                                              uint32_t &kmin, uint32_t &kmax)
{
    const float4 ra = scale4(va, ep.c_block);
    const float4 rb = scale4(vb, ep.c_block);
    if constexpr (RANGE) {
        if (ep.rotated != nullptr) {
            *reinterpret_cast<float4 *>(ep.rotated + j) = ra;
            *reinterpret_cast<float4 *>(ep.rotated + j + 4) = rb;
        }
        const float r[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const uint32_t key = float_key(r[e]);
            kmin = min(kmin, key);
            kmax = max(kmax, key);
        }
        return;
    }
    if (COMPRESS) {
        if (ep.rotated != nullptr) {
            *reinterpret_cast<float4 *>(ep.rotated + j) = ra;
            *reinterpret_cast<float4 *>(ep.rotated + j + 4) = rb;
        }
        const float r[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
        const uint4 rnd = round_call(j, ep.worker, ep.round, keys);
        const uint64_t z = quantize8<BITS, IDENTITY>(r, ep.kappa, ep.half_g, ep.gf, rnd, ep.lut);
        if constexpr (BITS == 8)
            *reinterpret_cast<uint2 *>(ep.packed + j) = make_uint2((uint32_t)z, (uint32_t)(z >> 32));
        else if constexpr (BITS == 4)
            *reinterpret_cast<uint32_t *>(ep.packed + j / 2) = (uint32_t)z;
        else if constexpr (BITS == 3)
            store_packed3(ep.packed, j, (uint32_t)z);
        else if constexpr (BITS == 2)
            *reinterpret_cast<uint16_t *>(ep.packed + j / 4) = (uint16_t)z;
        else
            ep.packed[j / 8] = (unsigned char)z;
    } else {
        if (j >= ep.d) return;
        const uint32_t bits = ep.sw[row * ep.words_per_row + (uu >> 2)] >> (uint32_t)(j & 31);
        float4 oa = flip4(ra, bits);
        float4 ob = flip4(rb, bits >> 4);
        if (j + 8 <= ep.d) {
            if (ep.xsub != nullptr) {
                const float4 xa = __ldcs(reinterpret_cast<const float4 *>(ep.xsub + j));
                const float4 xb = __ldcs(reinterpret_cast<const float4 *>(ep.xsub + j + 4));
                oa = make_float4(xa.x - oa.x, xa.y - oa.y, xa.z - oa.z, xa.w - oa.w);
                ob = make_float4(xb.x - ob.x, xb.y - ob.y, xb.z - ob.z, xb.w - ob.w);
            }
            *reinterpret_cast<float4 *>(ep.out + j) = oa;
            *reinterpret_cast<float4 *>(ep.out + j + 4) = ob;
        } else {
            const float o[8] = {oa.x, oa.y, oa.z, oa.w, ob.x, ob.y, ob.z, ob.w};
            for (int e = 0; e < 8; ++e)
                if (j + e < ep.d) ep.out[j + e] = ep.xsub != nullptr ? ep.xsub[j + e] - o[e] : o[e];
        }
    }
}

// Last round of a pass-B tile, any geometry: the top E row bits, each thread owning 2^E rows
// of one 8-coordinate unit, followed by the epilogue on the registers.
template <int E, bool COMPRESS, int BITS, bool IDENTITY, bool RANGE>
__device__ __forceinline__ void pass_b_last_round(const float4 *tile, int kb, int ccl, int tid, int mask,
                                                  const EpilogueCtx &ep, const PhiloxKeys &keys,
                                                  uint32_t &kmin, uint32_t &kmax)
{
    constexpr int N = 1 << E;
    const int ul = ccl - 1;                            // log2 units per row
    const int rl = kb - E;                             // log2 of the row stride of this round
#pragma unroll 1
    for (int i = 0; i < 8 / N; ++i) {
        const int gg = swap_bits_2_3(tid) + i * kPThreads;
        const int uu = gg & ((1 << ul) - 1);
        const int row_low = gg >> ul;
        float4 a[N], b[N];
#pragma unroll
        for (int m = 0; m < N; ++m) {
            const int c = ((row_low + (m << rl)) << ccl) + 2 * uu;
            a[m] = tile[c ^ ((c >> 3) & mask)];
            b[m] = tile[(c + 1) ^ ((c >> 3) & mask)];
        }
#pragma unroll
        for (int t = 0; t < E; ++t) {
#pragma unroll
            for (int m = 0; m < N; ++m)
                if (!(m & (1 << t))) {
                    butterfly(a[m], a[m | (1 << t)]);
                    butterfly(b[m], b[m | (1 << t)]);
                }
        }
        if constexpr (N == 8) {
            // eight rows: a loop of two iterations over four rows each, as in the 2^20 form
            // (the second iteration's rows move down the register arrays): half the code
#pragma unroll 1
            for (int half = 0; half < 2; ++half) {
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const int row = row_low + ((4 * half + m) << rl);
                    const uint64_t j = ep.j_tile + ((uint64_t)row << kPLog2) + 8 * uu;
                    epilogue_unit<COMPRESS, BITS, IDENTITY, RANGE>(a[m], b[m], j, row, uu, ep, keys, kmin, kmax);
                }
#pragma unroll
                for (int m = 0; m < 4; ++m) { a[m] = a[m + 4]; b[m] = b[m + 4]; }
            }
        } else {
#pragma unroll
            for (int m = 0; m < N; ++m) {
                const int row = row_low + (m << rl);
                const uint64_t j = ep.j_tile + ((uint64_t)row << kPLog2) + 8 * uu;
                epilogue_unit<COMPRESS, BITS, IDENTITY, RANGE>(a[m], b[m], j, row, uu, ep, keys, kmin, kmax);
            }
        }
    }
}

// The same for the k = 20 tile: two halves (columns 0-31, 32-63) of 128 rows x 8 chunks.
// Thread (u = tid & 3, rl from bits 2..5, h = tid >> 6) owns unit 4h + u of rows rl + 16 m,
// m = 0..7; lanes 0-7 of a quarter warp cover four units of two adjacent rows, whose XOR
// patterns differ in bit 0, so both chunk reads are conflict-free.
template <bool COMPRESS, int BITS, bool IDENTITY, bool RANGE>
__device__ __forceinline__ void pass_b_last_round_kb7(float4 *tile, int tid,
                                                      const EpilogueCtx &ep, const PhiloxKeys &keys,
                                                      uint32_t &kmin, uint32_t &kmax)
{
    const int u = tid & 3;
    const int rl = ((tid >> 2) & 1) | (((tid >> 3) & 7) << 1);
    const int h = tid >> 6;
    const int x = rl & 7;
    float4 *pa = tile + (h * 128 + rl) * 8 + ((2 * u) ^ x);
    float4 *pb = tile + (h * 128 + rl) * 8 + ((2 * u + 1) ^ x);
    {
        float4 a[8], b[8];
#pragma unroll
        for (int m = 0; m < 8; ++m) { a[m] = pa[m << 7]; b[m] = pb[m << 7]; }
#pragma unroll
        for (int t = 0; t < 3; ++t) {
#pragma unroll
            for (int m = 0; m < 8; ++m)
                if (!(m & (1 << t))) {
                    butterfly(a[m], a[m | (1 << t)]);
                    butterfly(b[m], b[m | (1 << t)]);
                }
        }
        // The epilogue is a loop of two iterations over four rows each (unrolled over all eight
        // it does not fit the instruction cache): the second iteration's rows move down the
        // register arrays in between.
        const int uu = 4 * h + u;
        const uint64_t j0 = ep.j_tile + ((uint64_t)rl << kPLog2) + 8 * uu;
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
#pragma unroll
            for (int m = 0; m < 4; ++m)
                epilogue_unit<COMPRESS, BITS, IDENTITY, RANGE>(a[m], b[m], j0 + ((uint64_t)(4 * half + m) << (kPLog2 + 4)),
                                                               rl + 16 * (4 * half + m), uu, ep, keys, kmin, kmax);
#pragma unroll
            for (int m = 0; m < 4; ++m) { a[m] = a[m + 4]; b[m] = b[m + 4]; }
        }
    }
}

// ------------------------------------------------------------------------------ the kernel
// KB = 7 specialises the k = 20 geometry at compile time; KB = 0 reads it from the params.
template <int MODE, int BITS, bool IDENTITY, int KB>
__global__ void __launch_bounds__(kPCtaThreads, 3)
thc_pipeline_kernel(const __grid_constant__ TmaMaps maps, PipeParams P, PtrArrayP in,
                    MutPtrArrayP outp, MutPtrArrayP rotated, PhiloxKeys keys)
{
    constexpr bool kFused = MODE == kCompressF32Fused;
    constexpr bool kEF = MODE == kErrorFeedback;
    constexpr bool kAgg = MODE == kAggDecompress;      // sums of table values formed in pass A
    constexpr bool kRange = MODE == kRangeF32;       // pass A as compress, epilogue = min / max
    constexpr bool kF32In = MODE == kCompressF32 || kFused || kRange;
    constexpr bool kCompress = kF32In || MODE == kCompressBF16;
    extern __shared__ __align__(1024) unsigned char pipe_smem_raw[];
    // TMA's 128-byte swizzle needs the tile buffers on 1024-byte boundaries of the shared
    // address space; the launch reserves 1 KB of slack for this round-up.
    unsigned char *pipe_smem = pipe_smem_raw +
        ((1024u - ((uint32_t)__cvta_generic_to_shared(pipe_smem_raw) & 1023u)) & 1023u);
    float4 *bufs[2] = {reinterpret_cast<float4 *>(pipe_smem),
                       reinterpret_cast<float4 *>(pipe_smem + kPElems * 4)};
    uint32_t *sw = reinterpret_cast<uint32_t *>(pipe_smem + 2 * kPElems * 4);
    unsigned char *lut = pipe_smem + 2 * kPElems * 4 + kPSignWords * 4;
    float2 *blk_const = reinterpret_cast<float2 *>(pipe_smem + 2 * kPElems * 4 + kPSignWords * 4 +
                                                   (size_t)(P.granularity + 1) * kLutEntryBytes);
    __shared__ TaskInfo s_info[2];
    __shared__ __align__(8) uint64_t s_mbar[2];
    __shared__ __align__(8) uint64_t s_done;           // one phase per finished task (compute warps arrive)
    __shared__ double s_sq[2][kPThreads / 32];          // fused scales: per-warp sums of squares of a tile

    const int tid = threadIdx.x;
    PipeCounters *pc = reinterpret_cast<PipeCounters *>(P.dev->counters);
    const int kb = KB ? KB : (int)P.kb;
    const uint32_t T = 1u << kb;                      // tiles (= panels) per worker-block
    const uint64_t B = 1ull << P.k;
    const int ccl = 11 - kb;                          // log2 chunks per pass-B row
    const int bmask = KB == 9 ? 3 : KB == 8 ? 7 : (int)P.b_swz_mask;   // swizzle of the pass-B tiles of the generic path
    const uint64_t d_rows32 = P.d >> 5;               // whole 32-coordinate rows of a gradient

    if (tid == 0) {
        mbar_init(&s_mbar[0], 1);
        mbar_init(&s_mbar[1], 1);
        mbar_init(&s_done, kPThreads);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (kCompress && !IDENTITY && !kRange) lut_fill<LutKind<BITS, IDENTITY>::k8>(lut, P.dev, P.granularity, tid, kPCtaThreads);
    // error feedback: table values as floats, one copy per lane (8 copies for 8-bit indices)
    constexpr int kFRep = BITS <= 4 ? 32 : 8;
    float *ftab = reinterpret_cast<float *>(lut);
    if (kEF) {
        for (int idx = tid; idx < (1 << BITS) * kFRep; idx += kPCtaThreads)
            ftab[idx] = (float)P.dev->table[idx / kFRep];
    }
    const uint32_t nblk_total = (uint32_t)(P.d_pad >> P.k);
    const uint32_t nblk_cached = nblk_total < (uint32_t)kBlockConstMax ? nblk_total : (uint32_t)kBlockConstMax;
    if (!kFused && !kRange) {
        for (uint32_t b = tid; b < nblk_cached; b += kPCtaThreads)
            blk_const[b] = block_constants<kCompress>(block_range(P.scales, b, P.nblocks, P.exact_range), P.granularity, P.divisor);
    }
    __syncthreads();

    if (tid >= kPThreads) {
        // ============================================================ control warp
        const int lane = tid - kPThreads;
        const uint64_t pol_stream = make_evict_first_policy();   // gradients: read once
        const uint64_t pol_ring = make_evict_normal_policy();    // ring: written and read in L2
        uint32_t uses[2] = {0u, 0u};                  // TMA loads issued per slot so far
        // The task last handed over in each slot whose completion is not yet signalled
        // (warp-uniform).  The control warp signals completions, so the release fence is off
        // the compute warps' critical path.  It learns of a finished task either from the
        // hand-shake (the compute warps picked up the next task) or, while it waits for a
        // dependency, from the s_done mbarrier: a dependency wait must never hold back the
        // signal of an earlier task, which may be the very thing waited for.
        TaskId pend[2];
        bool pend_valid[2] = {false, false};
        pend[0].wb = pend[0].idx = pend[0].is_b = pend[0].slot = pend[0].gen = 0;
        pend[1] = pend[0];

        // Warp-wide: publish the completion of task t (whose sums of squares sit in s_sq[sq]).
        // Fused scales: a pass-A tile is counted with a returning atomic; complete_issue only
        // issues it (lane 0 keeps the result, which nothing needs yet, so the claim of the next
        // task can be in flight at the same time) and complete_finish looks at it: the warp
        // that counted the last tile of an RHT block computes the block's M from the stored
        // sums (fixed order) and releases the block's pass-B tasks.
        auto complete_issue = [&](const TaskId &t, int sq, uint32_t &old, uint32_t &r) -> bool {
            if (!kFused || t.is_b) {
                if (lane == 0) red_release_add(t.is_b ? &pc->b_done[t.slot].v : &pc->a_done[t.slot].v, 1u);
                return false;
            }
            r = t.wb / P.n_local;
            old = 0;
            if (lane == 0) {
                const double tile_sum = (s_sq[sq][0] + s_sq[sq][1]) + (s_sq[sq][2] + s_sq[sq][3]);
                __stcg(P.tile_sq + (((size_t)t.wb << kb) + t.idx), tile_sum);
                old = atom_release_add(&pc->a_done[r & 15u].v, 1u);
            }
            return true;
        };
        auto complete_finish = [&](uint32_t old, uint32_t r) {
            old = __shfl_sync(0xFFFFFFFFu, old, 0);
            if (old + 1u != (r / 16u + 1u) * P.n_local * T) return;
            __threadfence();                           // the other tiles' sums, after seeing the count
            // Eight workers at a time, four lanes per worker: each lane adds every fourth of
            // its worker's T tile sums (all loads in flight together), the four lanes are
            // combined, one square root per worker, then the maximum over the workers.
            double ell = 0.0;
#pragma unroll 1
            for (uint32_t i0 = 0; i0 < P.n_local; i0 += 8u) {
                const uint32_t i = i0 + ((uint32_t)lane >> 2);
                const bool live = i < P.n_local;
                const double *p = P.tile_sq + ((size_t)(r * P.n_local + (live ? i : 0u)) << kb) + (lane & 3);
                double acc = 0.0;
#pragma unroll 8
                for (uint32_t c2 = 0; c2 < T; c2 += 4u) acc += __ldcg(p + c2);
                acc += __shfl_xor_sync(0xFFFFFFFFu, acc, 1);
                acc += __shfl_xor_sync(0xFFFFFFFFu, acc, 2);
                double norm = live ? sqrt(acc) : 0.0;
#pragma unroll
                for (int off = 4; off < 32; off <<= 1) {
                    const double other = __shfl_xor_sync(0xFFFFFFFFu, norm, off);
                    if (other > norm || other != other) norm = other;     // a NaN norm sticks
                }
                if (norm > ell || norm != norm) ell = norm;
            }
            if (lane == 0) {
                float M = (float)(P.t_p * ell / sqrt((double)B));
                uint32_t flags = 0;
                if (!isfinite(M)) { M = 0.0f; flags |= THC_STATUS_NONFINITE; }
                if (M == 0.0f) flags |= THC_STATUS_ZERO_BLOCK;
                __stcg(P.scales_out + r, M);
                // the quantiser's constants for the block's pass-B tasks (a division in fp64:
                // done once here instead of once per task)
                BlockRange br;
                br.hi = M; br.lo = -M;
                __stcg(P.fused_const + r, compress_constants(br));
                if (flags) atomicOr(&P.dev->status, flags);
                red_release_add(&pc->a_done[16u + (r & 15u)].v, 1u);
            }
        };
        auto complete = [&](const TaskId &t, int sq) {
            uint32_t old = 0, r = 0;
            if (complete_issue(t, sq, old, r)) complete_finish(old, r);
        };

        for (uint32_t i = 0;; ++i) {
            const int s = (int)(i & 1);
            // Task i is claimed once the compute warps have picked up task i-1, i.e. have
            // finished task i-2: buffer s and sign-word slot s are free.  One task of
            // look-ahead only: a deeper one stretches every task's claim-to-completion time,
            // which is what dependent tasks wait for.  Task i-2 is signalled first: task i
            // may depend on it.
            bool counting = false;
            uint32_t cnt_old = 0, cnt_r = 0;
            if (i >= 1) {
                bar_sync(3 + (s ^ 1), kPCtaThreads);
                if (pend_valid[s]) { counting = complete_issue(pend[s], s, cnt_old, cnt_r); pend_valid[s] = false; }
            }
            uint32_t q = 0, ab = 0;
            if (lane == 0) {
                q = atomicAdd(&pc->head, 1u);
                ab = ld_relaxed_u32(&pc->abort);
            }
            q = __shfl_sync(0xFFFFFFFFu, q, 0);
            ab = __shfl_sync(0xFFFFFFFFu, ab, 0);
            if (counting) complete_finish(cnt_old, cnt_r);
            bool have = (uint64_t)q < P.total_tasks && ab == 0;
            TaskId t;
            t.wb = t.idx = t.is_b = t.slot = t.gen = 0;
            uint32_t r = 0, tma = 0, phase = 0;            // tma, phase: lane 0
            if (have) {
                t = decode_task(q, P);
                r = t.wb / P.n_local;
                const uint32_t wl = t.wb - r * P.n_local;
                const uint64_t j0 = (uint64_t)r * B + ((uint64_t)t.idx << kPLog2);
                if (!t.is_b) {
                    // pass A reads only the caller's input: start the load before looking at
                    // the ring slot, which only the end of the task writes to
                    if (lane == 0 && kF32In && (j0 >> 5) + 256 <= d_rows32) {
                        mbar_expect_tx(&s_mbar[s], kPElems * 4);
                        tma_load_2d(bufs[s], &maps.in[wl], 0, (int)(j0 >> 5), &s_mbar[s], pol_stream);
                        tma = 1; phase = uses[s] & 1u; ++uses[s];
                    }
                    if (lane == 0 && MODE == kCompressBF16 && (j0 >> 5) + 256 <= d_rows32) {
                        mbar_expect_tx(&s_mbar[s], kPElems * 2);
                        tma_load_2d(bufs[s] + kPChunks / 2, &maps.in[wl], 0, (int)(j0 >> 5), &s_mbar[s], pol_stream);
                        tma = 1; phase = uses[s] & 1u; ++uses[s];
                    }
                    if (!kF32In && !(MODE == kCompressBF16 && (j0 >> 5) + 256 <= d_rows32)) {
                        // tiles the compute warps load themselves: pull the lines into L2 now
                        const uint32_t in_bits = MODE == kCompressBF16 ? 16u : MODE == kDecompress8 ? 8u
                                                 : MODE == kDecompress16 ? 16u : MODE == kDecompress32 ? 32u
                                                 : (uint32_t)BITS;
                        const uint64_t first = j0 * in_bits / 8;
                        const uint64_t limit = (MODE == kCompressBF16 ? P.d : P.d_pad) * in_bits / 8;
                        const uint32_t lines = (uint32_t)kPElems * in_bits / 8 / 128;
                        const uint32_t sources = kAgg ? P.agg_n : 1u;
                        for (uint32_t si = 0; si < sources; ++si) {
                            const unsigned char *src = static_cast<const unsigned char *>(in.p[kAgg ? si : (kEF || kCompress ? wl : 0)]);
                            for (uint32_t l = (uint32_t)lane; l < lines; l += 32u)
                                if (first + 128ull * l < limit) prefetch_l2(src + first + 128ull * l);
                        }
                    }
                    if (kCompress) {
                        // sign words of the tile (64 Philox calls, two per lane), while the copy is in flight
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            const int call = lane + 32 * c;
                            const uint4 ph = sign_call(j0 + 128ull * call, P.round, keys);
                            *reinterpret_cast<uint4 *>(sw + 256 * s + 4 * call) = ph;
                        }
                    }
                }
                // pass B needs its worker-block's tiles (fused scales: the block's M, which
                // implies them); pass A needs the previous tenant of its ring slot consumed
                const uint32_t *ctr = !t.is_b ? &pc->b_done[t.slot].v
                                      : kFused ? &pc->a_done[16u + (r & 15u)].v : &pc->a_done[t.slot].v;
                const uint32_t target = !t.is_b ? t.gen * T : kFused ? r / 16u + 1u : (t.gen + 1) * T;
                if (target != 0) {
                    have = false;
                    bool expired = true;
                    for (uint32_t it = 0; it < kMaxPolls; ++it) {
                        uint32_t v = 0, a2 = 0;
                        if (lane == 0) { v = ld_acquire_u32(ctr); a2 = ld_relaxed_u32(&pc->abort); }
                        v = __shfl_sync(0xFFFFFFFFu, v, 0);
                        a2 = __shfl_sync(0xFFFFFFFFu, a2, 0);
                        if (v >= target) { have = true; expired = false; break; }
                        if (a2 != 0) { expired = false; break; }
                        if (pend_valid[s ^ 1]) {               // task i-1 is phase i-1 of s_done
                            uint32_t fin = lane == 0 ? (uint32_t)mbar_test(&s_done, (uint32_t)(s ^ 1)) : 0u;
                            fin = __shfl_sync(0xFFFFFFFFu, fin, 0);
                            if (fin) { complete(pend[s ^ 1], s ^ 1); pend_valid[s ^ 1] = false; }
                        }
                        __nanosleep(it < 32 ? 20 : 200);
                    }
                    if (expired && lane == 0) {
                        atomicOr(&P.dev->status, THC_STATUS_WAIT_TIMEOUT);
                        atomicExch(&pc->abort, 1u);
                    }
                    // giving up with the tile's copy in flight: let it land before leaving
                    if (!have && lane == 0 && tma) (void)mbar_wait(&s_mbar[s], phase);
                }
            }
            TaskInfo ti;
            ti.idx = 0xFFFFFFFFu; ti.is_b = 0; ti.wl = 0; ti.r = 0; ti.slot = 0; ti.gen = 0; ti.tma = 0; ti.phase = 0;
            ti.bcx = 0.f; ti.bcy = 0.f;
            if (have) {
                ti.idx = t.idx;
                ti.is_b = t.is_b;
                ti.r = r;
                ti.wl = t.wb - r * P.n_local;
                ti.slot = t.slot;
                ti.gen = t.gen;
                pend[s] = t;
                pend_valid[s] = true;
                if (lane == 0 && t.is_b) {
                    if (kFused) {
                        ti.bcx = ld_relaxed_f32(&P.fused_const[r].x);
                        ti.bcy = ld_relaxed_f32(&P.fused_const[r].y);
                    }
                    // the ring was written through the generic proxy; the TMA unit reads it
                    fence_proxy_async_global();
                    if (KB == 7) {
                        // panel: 128 ring rows x 64 columns, as two boxes of 32 columns
                        mbar_expect_tx(&s_mbar[s], kPElems * 4);
                        const int x0 = (int)(t.idx << 6);
                        const int y0 = (int)(t.slot << 7);
                        tma_load_2d(bufs[s], &maps.ring, x0, y0, &s_mbar[s], pol_ring);
                        tma_load_2d(bufs[s] + 1024, &maps.ring, x0 + 32, y0, &s_mbar[s], pol_ring);
                        tma = 1; phase = uses[s] & 1u; ++uses[s];
                    } else if (P.b_tma == 3u) {
                        // k = 15 .. 19: 2^kb ring rows x 2^(13-kb) columns as one 3-D box
                        // (word, group of 32 columns, row); it lands in the run-time layout
                        mbar_expect_tx(&s_mbar[s], kPElems * 4);
                        tma_load_3d(bufs[s], &maps.ring, 0, (int)(t.idx << (8 - kb)), (int)(t.slot << kb),
                                    &s_mbar[s], pol_ring);
                        tma = 1; phase = uses[s] & 1u; ++uses[s];
                    } else if (P.b_tma) {
                        // k = 21: 256 ring rows x 32 columns, one box; k = 22: 512 rows x 16
                        // columns, two boxes of 256 rows
                        mbar_expect_tx(&s_mbar[s], kPElems * 4);
                        const int x0 = (int)(t.idx << (kPLog2 - kb));
                        const int y0 = (int)(t.slot << kb);
                        for (uint32_t bx = 0; bx < P.b_tma; ++bx)
                            tma_load_2d(bufs[s] + (kPChunks / P.b_tma) * bx, &maps.ring, x0, y0 + 256 * (int)bx,
                                        &s_mbar[s], pol_ring);
                        tma = 1; phase = uses[s] & 1u; ++uses[s];
                    }
                }
                if (t.is_b && kEF && KB == 7) {
                    // error feedback: the x values the epilogue will read (128 rows x 64 columns)
                    const uint64_t j_panel = (uint64_t)r * B + ((uint64_t)t.idx << 6);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint64_t jr = j_panel + ((uint64_t)(lane + 32 * c) << kPLog2);
                        const float *xr = static_cast<const float *>(rotated.p[t.wb - r * P.n_local]) + jr;
                        if (jr < P.d) prefetch_l2(xr);
                        if (jr + 32 < P.d) prefetch_l2(xr + 32);
                    }
                }
                ti.tma = tma;
                ti.phase = phase;
            }
            __syncwarp();
            if (lane == 0) s_info[s] = ti;
            __syncwarp();
            bar_arrive(1 + s, kPCtaThreads);                  // slot s is full
            if (!have) {
                // "no task" is picked up once task i-1 is finished: signal it, then leave.
                bar_sync(3 + s, kPCtaThreads);
                if (pend_valid[s ^ 1]) complete(pend[s ^ 1], s ^ 1);
                break;
            }
        }
    } else {
        // ============================================================ compute warps
        // Loads the control warp could not hand to the TMA unit (ragged last tile, bf16 or
        // summed inputs, run-time geometry): done here, synchronously.
        auto load_tile = [&](const TaskInfo &ti, float4 *tile) {
            const uint64_t policy = make_evict_first_policy();
            if (ti.is_b) {
                const float *src = P.ring + (size_t)ti.slot * B + ((size_t)ti.idx << (kPLog2 - kb));
#pragma unroll 4
                for (int i = 0; i < kPChunks / kPThreads; ++i) {
                    const int c = tid + i * kPThreads;
                    const int row = c >> ccl, cc = c & ((1 << ccl) - 1);
                    cp_async16(&tile[c ^ ((c >> 3) & bmask)], src + ((size_t)row << kPLog2) + 4 * cc);
                }
                return;
            }
            const uint64_t j0 = (uint64_t)ti.r * B + ((uint64_t)ti.idx << kPLog2);
            if (kF32In) {
                const float *x = static_cast<const float *>(in.p[ti.wl]);
#pragma unroll 4
                for (int i = 0; i < kPChunks / kPThreads; ++i) {
                    const int c = tid + i * kPThreads;
                    const uint64_t j = j0 + 4ull * c;
                    const uint32_t nbytes = j + 4 <= P.d ? 16u : j < P.d ? (uint32_t)(P.d - j) * 4u : 0u;
                    cp_async16_hint(&tile[pswz(c)], nbytes ? (const void *)(x + j) : (const void *)x,
                                    nbytes, policy);
                }
            } else if (MODE == kCompressBF16) {
                const uint16_t *x = static_cast<const uint16_t *>(in.p[ti.wl]);
#pragma unroll 2
                for (int i = 0; i < kPChunks / 2 / kPThreads; ++i) {
                    const int u = tid + i * kPThreads;
                    const uint64_t j = j0 + 8ull * u;
                    uint32_t w[4] = {0, 0, 0, 0};
                    if (j + 8 <= P.d) {
                        const uint4 q = __ldg(reinterpret_cast<const uint4 *>(x + j));
                        w[0] = q.x; w[1] = q.y; w[2] = q.z; w[3] = q.w;
                    } else {
                        for (int e = 0; e < 8; ++e)
                            if (j + e < P.d) w[e >> 1] |= (uint32_t)__ldg(x + j + e) << ((e & 1) * 16);
                    }
                    tile[pswz(2 * u)] = make_float4(__uint_as_float(w[0] << 16), __uint_as_float(w[0] & 0xFFFF0000u),
                                                    __uint_as_float(w[1] << 16), __uint_as_float(w[1] & 0xFFFF0000u));
                    tile[pswz(2 * u + 1)] = make_float4(__uint_as_float(w[2] << 16), __uint_as_float(w[2] & 0xFFFF0000u),
                                                        __uint_as_float(w[3] << 16), __uint_as_float(w[3] & 0xFFFF0000u));
                }
            }
        };

        // kAggDecompress with 4-bit indices and table values below 128: the table as 16 bytes
        uint32_t agg_tb[4] = {0u, 0u, 0u, 0u};
        uint32_t agg_chunk = 0;
        if (kAgg && BITS == 4 && P.granularity < 128u) {
#pragma unroll
            for (int q = 0; q < 4; ++q)
                agg_tb[q] = P.dev->table[4 * q] | (P.dev->table[4 * q + 1] << 8) | (P.dev->table[4 * q + 2] << 16) |
                            (P.dev->table[4 * q + 3] << 24);
            agg_chunk = 255u / P.granularity;
        }
        (void)agg_tb; (void)agg_chunk;
        bar_sync(1, kPCtaThreads);
        TaskInfo me = s_info[0];
        fence_proxy_async();
        bar_arrive(3, kPCtaThreads);

        for (uint32_t it = 0; me.idx != 0xFFFFFFFFu; ++it) {
            const int cur = (int)(it & 1);
            float4 *tile = bufs[cur];
            if (me.tma) {
                // Every thread waits for the tile itself, so no block barrier is needed here.
                // A load that never completes ends the launch: flag it and raise the abort
                // flag; this task then runs on whatever the buffer holds (addresses do not
                // depend on data) and the control warp claims nothing more.
                if (!mbar_wait(&s_mbar[cur], me.phase)) {
                    atomicOr(&P.dev->status, THC_STATUS_WAIT_TIMEOUT);
                    atomicExch(&pc->abort, 1u);
                }
            } else if (kCompress || me.is_b) {
                load_tile(me, tile);
                cp_async_commit();
                cp_async_wait_all();
                compute_barrier();
            }                                          // inverse pass A: round 1 fetches its own rows
            const bool is_b = me.is_b != 0;
            const uint32_t wl = me.wl;
            const uint64_t r = me.r;
            const uint32_t slot = me.slot;
            const uint32_t idx = me.idx;
            const float2 bc = kFused ? make_float2(me.bcx, me.bcy)
                              : kRange ? make_float2(0.f, 0.f)
                              : r < nblk_cached ? blk_const[r]
                                                : block_constants<kCompress>(block_range(P.scales, r, P.nblocks, P.exact_range), P.granularity, P.divisor);

            if (!is_b) {
                // ================================ pass A: tile idx of worker-block wb
                double sq = 0.0;
                if constexpr (MODE == kCompressBF16) {
                    const uint64_t j0 = r * B + ((uint64_t)idx << kPLog2);
                    (void)j0;
                    if (me.tma)
                        pass_a_round1_bf16(tile, sw + 256 * cur, tid);
                    else
                        pass_a_round1<true, false>(tile, sw + 256 * cur, tid);
                } else if constexpr (kCompress) {
                    sq = pass_a_round1<true, kFused>(tile, sw + 256 * cur, tid);
                } else if constexpr (kAgg) {
                    const size_t coord = r * B + ((uint64_t)idx << kPLog2);
                    pass_a_round1_aggregate(tile, in, P.agg_n, coord / 2, bc, outp.p[1], coord, P.agg_acc_bits, tid,
                                            agg_tb, agg_chunk);
                } else {
                    constexpr int kInBits = MODE == kDecompress8 ? 8 : MODE == kDecompress16 ? 16
                                            : MODE == kDecompress32 ? 32 : BITS;
                    const unsigned char *src = static_cast<const unsigned char *>(in.p[kEF ? wl : 0]) +
                        (r * B + ((uint64_t)idx << kPLog2)) * kInBits / 8;
                    pass_a_round1_inverse<MODE, BITS, kFRep>(tile, src, bc, ftab + (tid & (kFRep - 1)), tid);
                }
                if (kFused) {
                    for (int off = 16; off > 0; off >>= 1) sq += __shfl_xor_sync(0xFFFFFFFFu, sq, off);
                    if ((tid & 31) == 0) s_sq[cur][tid >> 5] = sq;
                }
                __syncwarp();                          // the next round stays inside the warp's rows
            } else if (KB == 7 && !kCompress) {
                // inverse transform, pass B: sign words of the panel's 128 rows x 64 columns, two
                // words of one Philox call per row and thread; the epilogue reads them after the
                // block barrier below.  (Slot `cur` was last read two tasks ago.)
                const uint64_t jr = r * B + ((uint64_t)idx << (kPLog2 - kb)) + ((uint64_t)tid << kPLog2);
                const uint4 ph = sign_call(jr, P.round, keys);
                const bool hi = ((jr >> 5) & 3u) != 0;         // words 2,3 of the call
                sw[256 * cur + 2 * tid] = hi ? ph.z : ph.x;
                sw[256 * cur + 2 * tid + 1] = hi ? ph.w : ph.y;
            }
            // The round on row bits 0..3 is the second round of every pass-A tile and the first
            // of a 2^20 block's pass-B panel: one copy of its code serves both.
            if (KB == 7 || !is_b) {
                round_rows_0_3(tile, tid);
                compute_barrier();
            }
            if (!is_b) {
                pass_a_round3_store(tile, P.ring + (size_t)slot * B + ((size_t)idx << kPLog2), tid);
            } else {
                // ================================ pass B: panel idx of worker-block wb
                const uint64_t j_tile = r * B + ((uint64_t)idx << (kPLog2 - kb));
                EpilogueCtx ep;
                ep.j_tile = j_tile;
                ep.kappa = bc.x; ep.half_g = bc.y; ep.gf = (float)P.granularity; ep.c_block = P.c_block;
                ep.lut = lut_lane_addr<LutKind<BITS, IDENTITY>::k8>(lut, tid);
                ep.worker = P.worker_base + wl; ep.round = P.round;
                ep.packed = kCompress ? static_cast<unsigned char *>(outp.p[wl]) : nullptr;
                ep.rotated = kCompress ? static_cast<float *>(rotated.p[wl]) : nullptr;
                ep.out = kCompress ? nullptr : static_cast<float *>(outp.p[wl]);
                ep.xsub = kEF ? static_cast<const float *>(rotated.p[wl]) : nullptr;
                ep.d = P.d;
                ep.sw = (!kCompress && KB == 7) ? sw + 256 * cur : sw;
                ep.words_per_row = max(1, (1 << (kPLog2 - kb)) >> 5);
                if (!kCompress && KB != 7) {
                    TileGeom g;
                    g.row_log2 = (uint32_t)kb; g.col_log2 = (uint32_t)(kPLog2 - kb);
                    g.row_stride = 1ull << kPLog2; g.round = P.round;
                    fill_sign_words(sw, g, j_tile, keys, tid, kPThreads);
                }
                const int e1 = kb < 4 ? kb : 4;
                if (KB != 7) {
                    switch (e1) {
                    case 4: p_round<4>(tile, ccl, tid, bmask); break;
                    case 3: p_round<3>(tile, ccl, tid, bmask); break;
                    default: p_round<2>(tile, ccl, tid, bmask); break;
                    }
                    compute_barrier();
                }
                uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
                if (KB == 7) {
                    pass_b_last_round_kb7<kCompress, BITS, IDENTITY, kRange>(tile, tid, ep, keys, kmin, kmax);
                } else {
                    const int rem = kb - e1;
                    const int e_last = rem < 3 ? rem : 3;
                    if (rem > e_last) p_rounds(tile, ccl + e1, ccl + kb - e_last, tid, bmask);
                    switch (e_last) {
                    case 3: pass_b_last_round<3, kCompress, BITS, IDENTITY, kRange>(tile, kb, ccl, tid, bmask, ep, keys, kmin, kmax); break;
                    case 2: pass_b_last_round<2, kCompress, BITS, IDENTITY, kRange>(tile, kb, ccl, tid, bmask, ep, keys, kmin, kmax); break;
                    case 1: pass_b_last_round<1, kCompress, BITS, IDENTITY, kRange>(tile, kb, ccl, tid, bmask, ep, keys, kmin, kmax); break;
                    default: pass_b_last_round<0, kCompress, BITS, IDENTITY, kRange>(tile, kb, ccl, tid, bmask, ep, keys, kmin, kmax); break;
                    }
                }
                if (kRange) {
                    kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
                    kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
                    if ((tid & 31) == 0) {
                        atomicMin(P.range_keys + r, kmin);
                        atomicMax(P.range_keys + P.nblocks + r, kmax);
                    }
                }
            }
            // Finished: tell the control warp (it signals the completion to the other CTAs),
            // then pick up the next task.  The block-wide barrier means every compute warp
            // has issued its stores and is done with the tile and the sign words.
            mbar_arrive(&s_done);
            bar_sync(1 + (cur ^ 1), kPCtaThreads);
            me = s_info[cur ^ 1];
            fence_proxy_async();
            bar_arrive(3 + (cur ^ 1), kPCtaThreads);
        }
    }
    __syncthreads();

    // ---- leave: the last CTA clears the counters for the next launch
    if (tid == 0) {
        __threadfence();
        const uint32_t left = atomicAdd(&pc->exited, 1u);
        if (left == gridDim.x - 1) {
            for (int sl = 0; sl < kMaxRing; ++sl) { pc->a_done[sl].v = 0; pc->b_done[sl].v = 0; }
            pc->abort = 0;
            pc->head = 0;
            __threadfence();
            pc->exited = 0;
        }
    }
}

}  // namespace thc
