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
// Each CTA keeps two tile buffers: while it computes task i from one, the tile of task i+1
// (claimed one task ahead, dependency polled early) streams into the other with cp.async.
//
// Counters (in the context's device block, all zero between launches; the last CTA to leave
// clears them):  head, exited, abort, a_done[R], b_done[R].  a_done[s] counts finished A tiles
// of slot s over the whole launch (generation g of the slot is complete at (g+1)*T),
// b_done[s] finished B panels (slot may be overwritten by generation g once it reaches g*T).
#pragma once
#include "thc_device.cuh"

namespace thc {

constexpr int kPLog2 = 13;                  // coordinates per pipeline tile
constexpr int kPElems = 1 << kPLog2;
constexpr int kPChunks = kPElems / 4;
constexpr int kPThreads = 128;                // compute threads of a CTA
constexpr int kPCtaThreads = 160;             // plus one control warp that runs the queue
constexpr int kPSignWords = 512;            // sign words a tile can need
constexpr int kMaxRing = 56;
constexpr int kBlockConstMax = 256;         // per-block constants cached in shared memory
constexpr uint32_t kMaxPolls = 1u << 21;

enum PipeMode { kCompressF32, kCompressBF16, kDecompress8, kDecompress16, kDecompress32 };

struct PipeCounters {          // layout inside DeviceBlock::counters
    uint32_t head;
    uint32_t exited;
    uint32_t abort;
    uint32_t pad;
    uint32_t a_done[kMaxRing];
    uint32_t b_done[kMaxRing];
};

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
    uint32_t loaded;           // dependency satisfied: its tile load may be / has been issued
    uint32_t pad;
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

// Bounded wait (one thread): true once *ctr >= target; false if the launch was aborted or
// the wait expired (then the timeout bit and the abort flag are set).
__device__ __forceinline__ bool wait_at_least(const uint32_t *ctr, uint32_t target,
                                              PipeCounters *pc, DeviceBlock *dev)
{
    for (uint32_t it = 0; it < kMaxPolls; ++it) {
        if (ld_acquire_u32(ctr) >= target) return true;
        if (ld_relaxed_u32(&pc->abort) != 0) return false;
        __nanosleep(it < 32 ? 20 : 200);
    }
    atomicOr(&dev->status, THC_STATUS_WAIT_TIMEOUT);
    atomicExch(&pc->abort, 1u);
    return false;
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
__device__ __forceinline__ void cp_async_wait_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

// Named barriers: 1,2 = task slot full; 3,4 = task slot consumed; 5 = compute warps only.
__device__ __forceinline__ void bar_sync(int id, int count)
{
    asm volatile("bar.sync %0, %1;" :: "r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_arrive(int id, int count)
{
    asm volatile("bar.arrive %0, %1;" :: "r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void compute_barrier() { bar_sync(5, kPThreads); }

// Barrier over the compute warps that also ORs a predicate: every thread gets the same answer.
__device__ __forceinline__ bool compute_barrier_or(bool pred)
{
    uint32_t out;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\t"
                 "barrier.cta.red.or.pred q, 5, %2, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                 : "=r"(out) : "r"((uint32_t)pred), "r"(kPThreads) : "memory");
    return out != 0;
}

__device__ __forceinline__ void red_release_add(uint32_t *p, uint32_t v)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}

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
__device__ __forceinline__ float2 block_constants(float M, uint32_t g, uint32_t divisor)
{
    float2 c = make_float2(0.f, 0.f);
    if (M > 0.0f && isfinite(M)) {
        if (COMPRESS) {
            c.x = (float)(1.0 / (2.0 * (double)M));
            c.y = 0.5f;
        } else {
            c.x = (float)(2.0 * (double)M / ((double)g * (double)divisor));
            c.y = -M;
        }
    }
    return c;
}

// ------------------------------------------------------------------ in-place tile rounds
// Butterfly stages on chunk-index bits [sp, sp+E) of a 2048-chunk tile (see fwht_round).
template <int E>
__device__ __forceinline__ void p_round(float4 *tile, int sp, int tid)
{
    constexpr int N = 1 << E;
    constexpr int kGroups = kPChunks >> E;
#pragma unroll 1
    for (int G = tid; G < kGroups; G += kPThreads) {
        const int low = G & ((1 << sp) - 1);
        const int base = ((G >> sp) << (sp + E)) | low;
        float4 v[N];
#pragma unroll
        for (int m = 0; m < N; ++m) v[m] = tile[swz(base + (m << sp))];
#pragma unroll
        for (int t = 0; t < E; ++t) {
#pragma unroll
            for (int m = 0; m < N; ++m)
                if (!(m & (1 << t))) butterfly(v[m], v[m | (1 << t)]);
        }
#pragma unroll
        for (int m = 0; m < N; ++m) tile[swz(base + (m << sp))] = v[m];
    }
}

__device__ __forceinline__ void p_rounds(float4 *tile, int lo, int hi, int tid)
{
    int sp = lo;
    while (sp < hi) {
        const int e = min(4, hi - sp);
        switch (e) {
        case 4: p_round<4>(tile, sp, tid); break;
        case 3: p_round<3>(tile, sp, tid); break;
        case 2: p_round<2>(tile, sp, tid); break;
        default: p_round<1>(tile, sp, tid); break;
        }
        sp += e;
        compute_barrier();
    }
}

// ------------------------------------------------------------------------------- pass A
// First round, in place: sign flip (compress), stages of stride 1 and 2 inside each chunk,
// then stride 4 .. 32 across the thread's 16 consecutive chunks.  Chunk 16*tid + m lives at
// 16*tid + (m ^ (tid & 7)).
template <bool FLIP>
__device__ __forceinline__ void pass_a_round1(float4 *tile, const uint32_t *sw, int tid)
{
    float4 *mine = tile + tid * 16;
    const int x = tid & 7;
    float4 v[16];
#pragma unroll
    for (int m = 0; m < 16; ++m) v[m] = mine[m ^ x];
    if (FLIP) {
        const uint2 w = *reinterpret_cast<const uint2 *>(sw + 2 * tid);
#pragma unroll
        for (int m = 0; m < 16; ++m)
            v[m] = flip4(v[m], (m < 8 ? w.x : w.y) >> ((m & 7) * 4));
    }
#pragma unroll
    for (int m = 0; m < 16; ++m) v[m] = stages01(v[m]);
#pragma unroll
    for (int t = 0; t < 4; ++t) {
#pragma unroll
        for (int m = 0; m < 16; ++m)
            if (!(m & (1 << t))) butterfly(v[m], v[m | (1 << t)]);
    }
#pragma unroll
    for (int m = 0; m < 16; ++m) mine[m ^ x] = v[m];
}

// Round on chunk bits 4..7 (also the first pass-B round when a row has 16 chunks): thread
// tid owns chunks hi*256 + 16*m + low (low = tid & 15, hi = tid >> 4), stored with the low
// three bits XORed by m & 7.
__device__ __forceinline__ void round_bits_4_7(float4 *tile, int tid)
{
    float4 *mine = tile + ((tid >> 4) << 8);
    const int low = tid & 15;
    float4 *q[8];
#pragma unroll
    for (int x = 0; x < 8; ++x) q[x] = mine + (low ^ x);
    float4 v[16];
#pragma unroll
    for (int m = 0; m < 16; ++m) v[m] = q[m & 7][16 * m];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
#pragma unroll
        for (int m = 0; m < 16; ++m)
            if (!(m & (1 << t))) butterfly(v[m], v[m | (1 << t)]);
    }
#pragma unroll
    for (int m = 0; m < 16; ++m) q[m & 7][16 * m] = v[m];
}

// Last round of a pass-A tile (chunk bits 8..10) with the result stored straight to the ring.
__device__ __forceinline__ void pass_a_round3_store(const float4 *tile, float *dst, int tid)
{
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int low = tid + i * kPThreads;
        const float4 *mine = tile + (low ^ ((low >> 4) & 7));
        float4 v[8];
#pragma unroll
        for (int m = 0; m < 8; ++m) v[m] = mine[m << 8];
#pragma unroll
        for (int t = 0; t < 3; ++t) {
#pragma unroll
            for (int m = 0; m < 8; ++m)
                if (!(m & (1 << t))) butterfly(v[m], v[m | (1 << t)]);
        }
        float4 *out = reinterpret_cast<float4 *>(dst) + low;
#pragma unroll
        for (int m = 0; m < 8; ++m) out[m << 8] = v[m];
    }
}

// ------------------------------------------------------------------------------- pass B
struct EpilogueCtx {
    uint64_t j_tile;        // coordinate of (row 0, column 0) of the tile in the worker's vector
    float kappa, half_g, gf, c_block;
    const uint4 *lut;
    uint32_t worker, round;
    unsigned char *packed;
    float *rotated;
    float *out;
    uint64_t d;
    const uint32_t *sw;
    int words_per_row;
};

template <bool COMPRESS, int BITS, bool IDENTITY>
__device__ __forceinline__ void epilogue_unit(const float4 &va, const float4 &vb, uint64_t j, int row,
                                              int uu, const EpilogueCtx &ep, const PhiloxKeys &keys)
{
    const float4 ra = scale4(va, ep.c_block);
    const float4 rb = scale4(vb, ep.c_block);
    if (COMPRESS) {
        if (ep.rotated != nullptr) {
            *reinterpret_cast<float4 *>(ep.rotated + j) = ra;
            *reinterpret_cast<float4 *>(ep.rotated + j + 4) = rb;
        }
        const float r[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
        const uint4 rnd = round_call(j, ep.worker, ep.round, keys);
        const uint64_t z = quantize8<BITS, IDENTITY>(r, ep.kappa, ep.half_g, ep.gf, rnd, ep.lut, kLutRep);
        if constexpr (BITS == 8)
            *reinterpret_cast<uint2 *>(ep.packed + j) = make_uint2((uint32_t)z, (uint32_t)(z >> 32));
        else if constexpr (BITS == 4)
            *reinterpret_cast<uint32_t *>(ep.packed + j / 2) = (uint32_t)z;
        else if constexpr (BITS == 2)
            *reinterpret_cast<uint16_t *>(ep.packed + j / 4) = (uint16_t)z;
        else
            ep.packed[j / 8] = (unsigned char)z;
    } else {
        if (j >= ep.d) return;
        const uint32_t bits = ep.sw[row * ep.words_per_row + (uu >> 2)] >> (uint32_t)(j & 31);
        const float4 oa = flip4(ra, bits);
        const float4 ob = flip4(rb, bits >> 4);
        if (j + 8 <= ep.d) {
            *reinterpret_cast<float4 *>(ep.out + j) = oa;
            *reinterpret_cast<float4 *>(ep.out + j + 4) = ob;
        } else {
            const float o[8] = {oa.x, oa.y, oa.z, oa.w, ob.x, ob.y, ob.z, ob.w};
            for (int e = 0; e < 8; ++e)
                if (j + e < ep.d) ep.out[j + e] = o[e];
        }
    }
}

// Last round of a pass-B tile, any geometry: the top E row bits, each thread owning 2^E rows
// of one 8-coordinate unit, followed by the epilogue on the registers.
template <int E, bool COMPRESS, int BITS, bool IDENTITY>
__device__ __forceinline__ void pass_b_last_round(const float4 *tile, int kb, int ccl, int tid,
                                                  const EpilogueCtx &ep, const PhiloxKeys &keys)
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
            a[m] = tile[swz(c)];
            b[m] = tile[swz(c + 1)];
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
#pragma unroll
        for (int m = 0; m < N; ++m) {
            const int row = row_low + (m << rl);
            const uint64_t j = ep.j_tile + ((uint64_t)row << kPLog2) + 8 * uu;
            epilogue_unit<COMPRESS, BITS, IDENTITY>(a[m], b[m], j, row, uu, ep, keys);
        }
    }
}

// The same for the 128-row x 16-chunk tile (k = 20): rows row_low + 16 m, m = 0..7; lanes
// 0-7 of a quarter warp cover four units of two adjacent rows, which is conflict-free.
template <bool COMPRESS, int BITS, bool IDENTITY>
__device__ __forceinline__ void pass_b_last_round_kb7(float4 *tile, int tid,
                                                      const EpilogueCtx &ep, const PhiloxKeys &keys)
{
    const int uu = (tid & 3) | ((tid >> 1) & 4);
    const int row_low = ((tid >> 2) & 1) | ((tid >> 4) << 1);
    const int x = row_low & 7;
    float4 *pa = tile + row_low * 16 + ((2 * uu) ^ x);
    float4 *pb = tile + row_low * 16 + ((2 * uu + 1) ^ x);
    {
        float4 a[8], b[8];
#pragma unroll
        for (int m = 0; m < 8; ++m) { a[m] = pa[m << 8]; b[m] = pb[m << 8]; }
#pragma unroll
        for (int t = 0; t < 3; ++t) {
#pragma unroll
            for (int m = 0; m < 8; ++m)
                if (!(m & (1 << t))) {
                    butterfly(a[m], a[m | (1 << t)]);
                    butterfly(b[m], b[m | (1 << t)]);
                }
        }
        // back to the thread's own slots: the epilogue below is a compact loop (code size)
#pragma unroll
        for (int m = 0; m < 8; ++m) { pa[m << 8] = a[m]; pb[m << 8] = b[m]; }
    }
    const uint64_t j0 = ep.j_tile + ((uint64_t)row_low << kPLog2) + 8 * uu;
#pragma unroll 2
    for (int m = 0; m < 8; ++m)
        epilogue_unit<COMPRESS, BITS, IDENTITY>(pa[m << 8], pb[m << 8], j0 + ((uint64_t)m << (kPLog2 + 4)),
                                                row_low + 16 * m, uu, ep, keys);
}

// ------------------------------------------------------------------------------ the kernel
// KB = 7 specialises the k = 20 geometry at compile time; KB = 0 reads it from the params.
template <int MODE, int BITS, bool IDENTITY, int KB>
__global__ void __launch_bounds__(kPCtaThreads, 3)
thc_pipeline_kernel(PipeParams P, PtrArrayP in, MutPtrArrayP outp, MutPtrArrayP rotated,
                    PhiloxKeys keys)
{
    constexpr bool kCompress = MODE == kCompressF32 || MODE == kCompressBF16;
    constexpr bool kAsyncA = MODE == kCompressF32;
    extern __shared__ __align__(1024) unsigned char pipe_smem[];
    float4 *bufs[2] = {reinterpret_cast<float4 *>(pipe_smem),
                       reinterpret_cast<float4 *>(pipe_smem + kPElems * 4)};
    uint32_t *sw = reinterpret_cast<uint32_t *>(pipe_smem + 2 * kPElems * 4);
    uint4 *lut = reinterpret_cast<uint4 *>(pipe_smem + 2 * kPElems * 4 + kPSignWords * 4);
    float2 *blk_const = reinterpret_cast<float2 *>(pipe_smem + 2 * kPElems * 4 + kPSignWords * 4 +
                                                   (size_t)(P.granularity + 1) * kLutRep * 16);
    __shared__ TaskInfo s_info[2];
    __shared__ uint32_t s_published;       // tasks the control warp has handed over so far

    const int tid = threadIdx.x;
    if (tid == 0) s_published = 0;
    PipeCounters *pc = reinterpret_cast<PipeCounters *>(P.dev->counters);
    const int kb = KB ? KB : (int)P.kb;
    const uint32_t T = 1u << kb;                      // tiles (= panels) per worker-block
    const uint64_t B = 1ull << P.k;
    const int ccl = 11 - kb;                          // log2 chunks per pass-B row
    const uint64_t policy = make_evict_first_policy();

    if (kCompress && !IDENTITY) {
        for (int idx = tid; idx < (int)(P.granularity + 1) * kLutRep; idx += kPThreads)
            lut[idx] = P.dev->lut[idx / kLutRep];
    }
    const uint32_t nblk_total = (uint32_t)(P.d_pad >> P.k);
    const uint32_t nblk_cached = nblk_total < (uint32_t)kBlockConstMax ? nblk_total : (uint32_t)kBlockConstMax;
    for (uint32_t b = tid; b < nblk_cached; b += kPThreads)
        blk_const[b] = block_constants<kCompress>(P.scales[b], P.granularity, P.divisor);
    __syncthreads();

    // ---- issue the tile load of a task into a buffer (all threads)
    auto issue_load = [&](const TaskInfo &ti, float4 *tile) {
        const bool is_b = ti.is_b != 0;
        const uint32_t wl = ti.wl;
        const uint64_t r = ti.r;
        const uint32_t slot = ti.slot;
        if (is_b) {
            // panel idx: rows 2^13 apart in the ring slot, 2^(13-kb) columns each
            const float *src = P.ring + (size_t)slot * B + ((size_t)ti.idx << (kPLog2 - kb));
            if (KB == 7) {
                // chunk tid + 128 i is (row (tid >> 4) + 8 i, column chunk tid & 15)
                const float *xs = src + ((size_t)(tid >> 4) << kPLog2) + 4 * (tid & 15);
                float4 *dst = tile + (tid ^ ((tid >> 4) & 7));
#pragma unroll
                for (int i = 0; i < kPChunks / kPThreads; ++i)
                    cp_async16(dst + i * kPThreads, xs + ((size_t)i << (kPLog2 + 3)));
            } else
#pragma unroll 4
            for (int i = 0; i < kPChunks / kPThreads; ++i) {
                const int c = tid + i * kPThreads;
                const int row = c >> ccl, cc = c & ((1 << ccl) - 1);
                cp_async16(&tile[swz(c)], src + ((size_t)row << kPLog2) + 4 * cc);
            }
        } else {
            const uint64_t j0 = r * B + ((uint64_t)ti.idx << kPLog2);
            if (kAsyncA) {
                const float *x = static_cast<const float *>(in.p[wl]);
                if (j0 + kPElems <= P.d) {
                    const float *xs = x + j0 + 4 * tid;
                    float4 *dst = tile + (tid ^ ((tid >> 4) & 7));
#pragma unroll
                    for (int i = 0; i < kPChunks / kPThreads; ++i)
                        cp_async16_hint(dst + i * kPThreads, xs + 4 * i * kPThreads, 16u, policy);
                } else {
#pragma unroll 4
                    for (int i = 0; i < kPChunks / kPThreads; ++i) {
                        const int c = tid + i * kPThreads;
                        const uint64_t j = j0 + 4ull * c;
                        const uint32_t nbytes = j + 4 <= P.d ? 16u : j < P.d ? (uint32_t)(P.d - j) * 4u : 0u;
                        cp_async16_hint(&tile[swz(c)], nbytes ? (const void *)(x + j) : (const void *)x,
                                        nbytes, policy);
                    }
                }
            } else if (MODE == kCompressBF16) {
                const uint16_t *x = static_cast<const uint16_t *>(in.p[wl]);
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
                    tile[swz(2 * u)] = make_float4(__uint_as_float(w[0] << 16), __uint_as_float(w[0] & 0xFFFF0000u),
                                                   __uint_as_float(w[1] << 16), __uint_as_float(w[1] & 0xFFFF0000u));
                    tile[swz(2 * u + 1)] = make_float4(__uint_as_float(w[2] << 16), __uint_as_float(w[2] & 0xFFFF0000u),
                                                       __uint_as_float(w[3] << 16), __uint_as_float(w[3] & 0xFFFF0000u));
                }
            } else {
                constexpr int kPer = MODE == kDecompress8 ? 16 : MODE == kDecompress16 ? 8 : 4;
                const unsigned char *y = static_cast<const unsigned char *>(in.p[0]);
                const float2 bc = r < nblk_cached ? blk_const[r]
                                                  : block_constants<false>(P.scales[r], P.granularity, P.divisor);
#pragma unroll 2
                for (int i = 0; i < kPElems / kPer / kPThreads; ++i) {
                    const int u = tid + i * kPThreads;
                    const uint64_t j = j0 + (uint64_t)u * kPer;
                    const uint4 q = __ldg(reinterpret_cast<const uint4 *>(y + j * (16 / kPer)));
                    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                    for (int cc = 0; cc < kPer / 4; ++cc) {
                        float s[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int ix = cc * 4 + e;
                            uint32_t val;
                            if (MODE == kDecompress8) val = (w[ix >> 2] >> ((ix & 3) * 8)) & 0xFFu;
                            else if (MODE == kDecompress16) val = (w[ix >> 1] >> ((ix & 1) * 16)) & 0xFFFFu;
                            else val = w[ix];
                            const float yf = MODE == kDecompress32 ? (float)val
                                             : __uint_as_float(0x4B000000u | val) - 8388608.0f;
                            s[e] = fmaf(yf, bc.x, bc.y);
                        }
                        tile[swz(u * (kPer / 4) + cc)] = make_float4(s[0], s[1], s[2], s[3]);
                    }
                }
            }
        }
    };

    // ================================================================ control warp
    // Lane 0 claims tasks, waits (bounded) for their dependency and hands them to the compute
    // warps through s_info[0/1]; it runs at most two tasks ahead of them.
    if (tid >= kPThreads) {
        const int lane = tid - kPThreads;
        for (uint32_t i = 0;; ++i) {
            const int s = (int)(i & 1);
            TaskInfo ti;
            ti.idx = 0xFFFFFFFFu; ti.is_b = 0; ti.wl = 0; ti.r = 0; ti.slot = 0; ti.gen = 0; ti.loaded = 0; ti.pad = 0;
            // claim task i only once the compute warps have picked up task i-1: a deeper
            // look-ahead would stretch every task's claim-to-completion time, which is what
            // dependent tasks wait for
            if (i >= 1) bar_sync(3 + (s ^ 1), kPCtaThreads);
            if (lane == 0) {
                const uint32_t q = atomicAdd(&pc->head, 1u);
                if ((uint64_t)q < P.total_tasks) {
                    const TaskId t = decode_task(q, P);
                    const uint32_t *ctr = t.is_b ? &pc->a_done[t.slot] : &pc->b_done[t.slot];
                    const uint32_t target = t.is_b ? (t.gen + 1) * T : t.gen * T;
                    if (target == 0 || wait_at_least(ctr, target, pc, P.dev)) {
                        ti.idx = t.idx;
                        ti.is_b = t.is_b;
                        ti.r = t.wb / P.n_local;
                        ti.wl = t.wb - ti.r * P.n_local;
                        ti.slot = t.slot;
                        ti.gen = t.gen;
                        ti.loaded = 1;
                    }
                }
            }
            __syncwarp();
            if (lane == 0) {
                s_info[s] = ti;
                __threadfence_block();
                *reinterpret_cast<volatile uint32_t *>(&s_published) = i + 1;
            }
            __syncwarp();
            bar_arrive(1 + s, kPCtaThreads);                  // slot s is full
            if (__shfl_sync(0xFFFFFFFFu, ti.idx, 0) == 0xFFFFFFFFu) break;
        }
    } else {
    // ================================================================ compute warps
    bar_sync(1, kPCtaThreads);
    TaskInfo me = s_info[0];
    bar_arrive(3, kPCtaThreads);
    bool me_loaded = false;

    for (uint32_t it = 0; me.idx != 0xFFFFFFFFu; ++it) {
        const int cur = (int)(it & 1);
        const int s1 = cur ^ 1;
        if (!me_loaded) issue_load(me, bufs[cur]);
        cp_async_commit();
        cp_async_wait_all();
        // Every barrier of the task doubles as a look at the hand-over flag: as soon as the
        // control warp has published the next task, its tile starts streaming into the other
        // buffer.  A task is never waited for before the current one is finished and
        // signalled: it may depend on it.
        bool have_next = false;
        TaskInfo nxt = me;
        auto barrier_and_prefetch = [&]() {
            const bool pub = compute_barrier_or(
                !have_next && *reinterpret_cast<volatile uint32_t *>(&s_published) >= it + 2);
            if (pub) {
                bar_sync(1 + s1, kPCtaThreads);
                nxt = s_info[s1];
                bar_arrive(3 + s1, kPCtaThreads);
                if (nxt.idx != 0xFFFFFFFFu) issue_load(nxt, bufs[s1]);
                cp_async_commit();
                have_next = true;
            }
        };

        const bool is_b = me.is_b != 0;
        const uint32_t wl = me.wl;
        const uint64_t r = me.r;
        const uint32_t slot = me.slot;
        const uint32_t idx = me.idx;
        float4 *tile = bufs[cur];
        const float2 bc = r < nblk_cached ? blk_const[r]
                                          : block_constants<kCompress>(P.scales[r], P.granularity, P.divisor);

        if (!is_b) {
            // ================================ pass A: tile idx of worker-block wb
            const uint64_t j0 = r * B + ((uint64_t)idx << kPLog2);
            if (kCompress && tid < 64) {               // sign words of the tile: 64 calls
                const uint4 ph = sign_call(j0 + 128ull * tid, P.round, keys);
                *reinterpret_cast<uint4 *>(sw + 4 * tid) = ph;
            }
            barrier_and_prefetch();                   // tile and sign words visible
            pass_a_round1<kCompress>(tile, sw, tid);
            barrier_and_prefetch();
            round_bits_4_7(tile, tid);
            barrier_and_prefetch();
            pass_a_round3_store(tile, P.ring + (size_t)slot * B + ((size_t)idx << kPLog2), tid);
        } else {
            // ================================ pass B: panel idx of worker-block wb
            const uint64_t j_tile = r * B + ((uint64_t)idx << (kPLog2 - kb));
            EpilogueCtx ep;
            ep.j_tile = j_tile;
            ep.kappa = bc.x; ep.half_g = bc.y; ep.gf = (float)P.granularity; ep.c_block = P.c_block;
            ep.lut = lut + (tid & (kLutRep - 1));
            ep.worker = P.worker_base + wl; ep.round = P.round;
            ep.packed = kCompress ? static_cast<unsigned char *>(outp.p[wl]) : nullptr;
            ep.rotated = kCompress ? static_cast<float *>(rotated.p[wl]) : nullptr;
            ep.out = kCompress ? nullptr : static_cast<float *>(outp.p[0]);
            ep.d = P.d;
            ep.sw = sw;
            ep.words_per_row = max(1, (1 << (kPLog2 - kb)) >> 5);
            if (!kCompress) {
                TileGeom g;
                g.row_log2 = (uint32_t)kb; g.col_log2 = (uint32_t)(kPLog2 - kb);
                g.row_stride = 1ull << kPLog2; g.round = P.round;
                fill_sign_words(sw, g, j_tile, keys, tid, kPThreads);
            }
            barrier_and_prefetch();                   // tile (and sign words) visible
            const int e1 = kb < 4 ? kb : 4;
            if (KB == 7) {
                round_bits_4_7(tile, tid);
            } else {
                switch (e1) {
                case 4: p_round<4>(tile, ccl, tid); break;
                case 3: p_round<3>(tile, ccl, tid); break;
                default: p_round<2>(tile, ccl, tid); break;
                }
            }
            barrier_and_prefetch();
            if (KB == 7) {
                pass_b_last_round_kb7<kCompress, BITS, IDENTITY>(tile, tid, ep, keys);
            } else {
                const int rem = kb - e1;
                const int e_last = rem < 3 ? rem : 3;
                if (rem > e_last) p_rounds(tile, ccl + e1, ccl + kb - e_last, tid);
                switch (e_last) {
                case 3: pass_b_last_round<3, kCompress, BITS, IDENTITY>(tile, kb, ccl, tid, ep, keys); break;
                case 2: pass_b_last_round<2, kCompress, BITS, IDENTITY>(tile, kb, ccl, tid, ep, keys); break;
                case 1: pass_b_last_round<1, kCompress, BITS, IDENTITY>(tile, kb, ccl, tid, ep, keys); break;
                default: pass_b_last_round<0, kCompress, BITS, IDENTITY>(tile, kb, ccl, tid, ep, keys); break;
                }
            }
        }
        // every compute warp has issued its stores and is done with the tile and sign words
        compute_barrier();
        if (tid == 0) red_release_add(is_b ? &pc->b_done[slot] : &pc->a_done[slot], 1u);
        if (!have_next) {
            bar_sync(1 + s1, kPCtaThreads);
            nxt = s_info[s1];
            bar_arrive(3 + s1, kPCtaThreads);
        }
        me_loaded = have_next;
        me = nxt;
    }
    cp_async_wait_all();
    }
    __syncthreads();

    // ---- leave: the last CTA clears the counters for the next launch
    if (tid == 0) {
        __threadfence();
        const uint32_t left = atomicAdd(&pc->exited, 1u);
        if (left == gridDim.x - 1) {
            for (int s = 0; s < kMaxRing; ++s) { pc->a_done[s] = 0; pc->b_done[s] = 0; }
            pc->abort = 0;
            pc->head = 0;
            __threadfence();
            pc->exited = 0;
        }
    }
}

}  // namespace thc
