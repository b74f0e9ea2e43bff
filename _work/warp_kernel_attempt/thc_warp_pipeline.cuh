// Persistent dataflow kernel for the 2^20-coordinate RHT block (the paper's 4 MB partition,
// Section 2.1), fp32 gradients in, packed indices out: thc_compress and thc_prepare_compress.
//
// Same two-pass task graph, queue, ring and counters as thc_pipeline_kernel (see
// thc_pipeline.cuh): A(wb, t) transforms 2^13 consecutive coordinates (strides 1 .. 2^11) and
// writes them to the ring slot of worker-block wb; B(wb, p) transforms a panel of 256 rows
// (2^12 coordinates apart) x 32 columns (strides 2^12 .. 2^19) and runs the quantiser.  What
// differs is how a CTA runs its tasks:
//
//   * A thread holds 32 chunks of 16 bytes (128 registers of data), so a warp owns 4096
//     coordinates and five butterfly stages fit one round: the 20 stages take four trips
//     through shared memory (2+5 and 5 in pass A, 5 and 3 in pass B) instead of five, and the
//     epilogue runs from the registers of the last round.
//   * Pass A needs no synchronisation beyond the warp: each of the two warps of a pair owns
//     one half of the task's tile.  Pass B needs one 64-thread barrier between its rounds.
//   * One CTA per SM: a producer warp and four consumer pairs around a ring of six (five for
//     large tables) 32 KB tile buffers.  The producer claims tasks from the global queue,
//     waits for their dependencies, has the TMA unit fill the next free buffer, publishes a
//     descriptor and signals finished tasks to the other CTAs; pair p takes the buffers
//     p, p + 4, p + 8, ... of the fill sequence.  Up to two buffers are in flight while four
//     are being worked on.
//
// Shared-memory layouts (16-byte chunk index c of a 4096-coordinate half tile, 10 bits):
//   pass A   row rho = (c[3:4] << 5) | c[5:9] of 128 bytes, slot c[0:2] ^ (rho & 7): four TMA
//            boxes of 32 rows taken 4 gradient rows apart.  Round 1 (lane = c[5:9], thread
//            holds c[0:4]) and round 2 (lane = c[0:4], thread holds c[5:9]) are both
//            conflict-free for 128-bit accesses.
//   pass B   row t (256 rows), slot q (8 slots = 32 columns) at q ^ (t & 7): one TMA box.
//            Round 1: warp = t7, lane = (q, t5, t6), thread holds t0..t4; round 2: warp = q2,
//            lane = t0..t4, thread holds (t5, t6, t7) x (q0, q1).
// Every wait is bounded (see thc_pipeline.cuh); on expiry THC_STATUS_WAIT_TIMEOUT is set, the
// abort flag ends all CTAs and the kernel returns.
#pragma once
#include "thc_pipeline.cuh"

namespace thc {

constexpr int kWPairs = 4;                        // consumer pairs per CTA
constexpr int kWThreads = 32 + 64 * kWPairs;      // producer warp + consumers
constexpr int kWMaxBuf = 6;                       // tile buffers of 32 KB
constexpr int kWBufBytes = 32768;

struct WarpMaps {                                 // one 3-D map per worker gradient, one 2-D map for the ring
    CUtensorMap in[THC_MAX_WORKERS];
    CUtensorMap ring;
};

struct WarpDesc {                                 // published by the producer with each filled buffer
    uint32_t idx;                                 // tile / panel index
    uint32_t is_b;
    uint32_t wl;                                  // local worker
    uint32_t r;                                   // RHT block
    uint32_t slot;                                // ring slot
    uint32_t tma;                                 // the tile was filled by TMA (else the consumers load it)
    uint32_t end;                                 // no task: the pair leaves
    float    bcx, bcy;                            // block constants of a pass-B task
};

__device__ __forceinline__ void mbar_expect_tx_only(uint64_t *bar, uint32_t bytes)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(bar);
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" :: "r"(a), "r"(bytes) : "memory");
}

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

// Butterfly stages on bits [first, first + NB) of the index of a thread's 32 chunks.
template <int NB>
__device__ __forceinline__ void stages32(float4 (&v)[32], int first)
{
#pragma unroll
    for (int t = first; t < first + NB; ++t) {
#pragma unroll
        for (int m = 0; m < 32; ++m)
            if (!(m & (1 << t))) butterfly(v[m], v[m | (1 << t)]);
    }
}

// Packed indices of two adjacent units (16 coordinates from j, j a multiple of 16).
template <int BITS>
__device__ __forceinline__ void store_packed_pair(unsigned char *pk, uint64_t j, uint64_t z0, uint64_t z1)
{
    if constexpr (BITS == 8) {
        *reinterpret_cast<uint4 *>(pk + j) = make_uint4((uint32_t)z0, (uint32_t)(z0 >> 32), (uint32_t)z1, (uint32_t)(z1 >> 32));
    } else if constexpr (BITS == 4) {
        *reinterpret_cast<uint2 *>(pk + j / 2) = make_uint2((uint32_t)z0, (uint32_t)z1);
    } else if constexpr (BITS == 3) {
        const uint64_t w = (z0 & 0xFFFFFFull) | ((z1 & 0xFFFFFFull) << 24);     // 48 bits at byte 3 j / 8
        uint16_t *p = reinterpret_cast<uint16_t *>(pk + 3 * (j >> 3));
        p[0] = (uint16_t)w; p[1] = (uint16_t)(w >> 16); p[2] = (uint16_t)(w >> 32);
    } else if constexpr (BITS == 2) {
        *reinterpret_cast<uint32_t *>(pk + j / 4) = ((uint32_t)z0 & 0xFFFFu) | ((uint32_t)z1 << 16);
    } else {
        *reinterpret_cast<uint16_t *>(pk + j / 8) = (uint16_t)(((uint32_t)z0 & 0xFFu) | ((uint32_t)z1 << 8));
    }
}

template <int BITS, bool IDENTITY>
__global__ void __launch_bounds__(kWThreads, 1)
thc_warp_pipeline_kernel(const __grid_constant__ WarpMaps maps, PipeParams P, PtrArrayP in,
                         MutPtrArrayP outp, MutPtrArrayP rotated, PhiloxKeys keys)
{
    constexpr bool kLut8 = LutKind<BITS, IDENTITY>::k8;
    extern __shared__ __align__(1024) unsigned char wp_smem_raw[];
    unsigned char *smem = wp_smem_raw +
        ((1024u - ((uint32_t)__cvta_generic_to_shared(wp_smem_raw) & 1023u)) & 1023u);
    constexpr int nbuf = kWMaxBuf;
    unsigned char *lut = smem + (size_t)nbuf * kWBufBytes;
    float2 *blk_const = reinterpret_cast<float2 *>(lut + (size_t)(P.granularity + 1) * 128);   // first kBlockConstMax blocks
    __shared__ WarpDesc s_desc[kWMaxBuf];
    __shared__ __align__(8) uint64_t s_full[kWMaxBuf];      // buffer filled and described (producer + TMA bytes)
    __shared__ __align__(8) uint64_t s_done[kWMaxBuf];      // task finished (one arrival per consumer warp)
    __shared__ __align__(8) uint64_t s_pair[kWPairs];       // the two warps of a pair between the rounds of pass B
    __shared__ uint32_t s_fills[kWMaxBuf];                  // fills of each buffer published so far

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    PipeCounters *pc = reinterpret_cast<PipeCounters *>(P.dev->counters);
    constexpr uint32_t T = 128;                       // tasks per worker-block and pass
    const uint64_t B = 1ull << 20;

    if (tid == 0) {
        for (int b = 0; b < kWMaxBuf; ++b) { mbar_init(&s_full[b], 1); mbar_init(&s_done[b], 2); }
        for (int p = 0; p < kWPairs; ++p) mbar_init(&s_pair[p], 2);
        for (int b = 0; b < kWMaxBuf; ++b) s_fills[b] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (!IDENTITY) lut_fill<kLut8>(lut, P.dev, P.granularity, tid, kWThreads);
    const uint32_t nblk_cached = P.nblocks < (uint32_t)kBlockConstMax ? P.nblocks : (uint32_t)kBlockConstMax;
    for (uint32_t bk = tid; bk < nblk_cached; bk += kWThreads)
        blk_const[bk] = compress_constants(block_range(P.scales, bk, P.nblocks, P.exact_range));
    __syncthreads();

    if (warp == 0) {
        // ================================================================ producer warp
        // Lane b < nbuf runs buffer b through  free -> claimed (waiting for the task's dependency)
        // -> busy (handed to a consumer pair) -> free;  the lanes work side by side, so the global
        // round trips of up to nbuf tasks (claim, dependency poll, completion signal) overlap.
        // Queue positions are claimed for the free buffers that come next in the fill sequence,
        // one atomic for all of them and in that order: a CTA therefore hands its tasks to its
        // pairs in queue order, and a task never waits for one that the same pair runs later.
        const uint64_t pol_stream = make_evict_first_policy();   // gradients: read once
        const uint64_t pol_ring = make_evict_normal_policy();    // ring: written and read in L2
        enum { kFree = 0, kClaimed = 1, kBusy = 2 };
        int state = kFree;
        uint32_t uses = 0;                              // fills of this lane's buffer so far
        uint32_t done_par = 0;
        TaskId t;
        t.wb = t.idx = t.is_b = t.slot = t.gen = 0;
        uint32_t t_r = 0, t_wl = 0, t_tma = 0, polls = 0;
        bool end_sent = false;
        uint32_t fill = 0;                              // next index of the fill sequence (warp-uniform)
        bool finished = false;                          // warp-uniform: no more claims
        const uint64_t d_rows128 = P.d >> 7;            // whole groups of four 32-coordinate rows
        unsigned char *buf = smem + (size_t)(lane < nbuf ? lane : 0) * kWBufBytes;
        const bool owner = lane < nbuf;

        auto publish_end = [&]() {
            WarpDesc e;
            e.idx = 0; e.is_b = 0; e.wl = 0; e.r = 0; e.slot = 0; e.tma = 0; e.end = 1; e.bcx = 0.f; e.bcy = 0.f;
            s_desc[lane] = e;
            ++uses;
            *reinterpret_cast<volatile uint32_t *>(&s_fills[lane]) = uses;
            mbar_arrive(&s_full[lane]);
            end_sent = true;
        };

        for (uint32_t idle = 0;;) {
            bool progress = false;
            // ---- 1. finished tasks: tell the other CTAs
            if (owner && state == kBusy && mbar_test(&s_done[lane], done_par)) {
                red_release_add(t.is_b ? &pc->b_done[t.slot].v : &pc->a_done[t.slot].v, 1u);
                state = kFree;
                done_par ^= 1u;
                progress = true;
            }
            // ---- 2. claim queue positions for the run of free buffers that comes next
            const uint32_t free_mask = __ballot_sync(0xFFFFFFFFu, owner && state == kFree && !end_sent);
            if (!finished) {
                uint32_t m = 0;
                while (m < (uint32_t)nbuf && ((free_mask >> ((fill + m) % (uint32_t)nbuf)) & 1u)) ++m;
                if (m > 0) {
                    uint32_t base = 0, ab = 0;
                    if (lane == 0) {
                        base = atomicAdd(&pc->head, m);
                        ab = ld_relaxed_u32(&pc->abort);
                    }
                    base = __shfl_sync(0xFFFFFFFFu, base, 0);
                    ab = __shfl_sync(0xFFFFFFFFu, ab, 0);
                    const uint32_t rank = ((uint32_t)lane + (uint32_t)nbuf - fill % (uint32_t)nbuf) % (uint32_t)nbuf;
                    if (owner && rank < m) {
                        const uint32_t q = base + rank;
                        if ((uint64_t)q < P.total_tasks && ab == 0) {
                            t = decode_task(q, P);
                            t_r = t.wb / P.n_local;
                            t_wl = t.wb - t_r * P.n_local;
                            t_tma = 0;
                            polls = 0;
                            if (!t.is_b) {
                                // pass A reads only the caller's input: start the load before looking
                                // at the ring slot, which only the end of the task writes to
                                const uint64_t j0 = (uint64_t)t_r * B + ((uint64_t)t.idx << kPLog2);
                                if ((j0 >> 7) + 64 <= d_rows128) {
                                    fence_proxy_async();
                                    mbar_expect_tx_only(&s_full[lane], kWBufBytes);
#pragma unroll 1
                                    for (int bx = 0; bx < 8; ++bx)      // half bx >> 2, every fourth row from bx & 3
                                        tma_load_3d(buf + (bx >> 2) * 16384 + (bx & 3) * 4096, &maps.in[t_wl], 0, bx & 3,
                                                    (int)((j0 >> 7) + (uint64_t)(bx >> 2) * 32u), &s_full[lane], pol_stream);
                                    t_tma = 1;
                                }
                            }
                            state = kClaimed;
                        }
                    }
                    fill += m;
                    if ((uint64_t)(base + m) > P.total_tasks || ab != 0) finished = true;
                    progress = true;
                }
            }
            // ---- 3. claimed tasks: once the dependency holds, fill (pass B) and hand over.
            // Pass B needs its worker-block's tiles; pass A needs the previous tenant of its ring
            // slot consumed.
            if (owner && state == kClaimed) {
                const uint32_t *ctr = !t.is_b ? &pc->b_done[t.slot].v : &pc->a_done[t.slot].v;
                const uint32_t target = !t.is_b ? t.gen * T : (t.gen + 1) * T;
                bool ready = target == 0;
                bool give_up = false;
                if (!ready) {
                    ready = ld_acquire_u32(ctr) >= target;
                    if (!ready) {
                        give_up = ld_relaxed_u32(&pc->abort) != 0;
                        if (++polls > kMaxPolls) {
                            atomicOr(&P.dev->status, THC_STATUS_WAIT_TIMEOUT);
                            atomicExch(&pc->abort, 1u);
                            give_up = true;
                        }
                    }
                }
                if (ready) {
                    WarpDesc e;
                    e.idx = t.idx; e.is_b = t.is_b; e.wl = t_wl; e.r = t_r; e.slot = t.slot; e.tma = t_tma; e.end = 0;
                    e.bcx = 0.f; e.bcy = 0.f;
                    if (t.is_b) {
                        const float2 c = t_r < nblk_cached ? blk_const[t_r]
                                                           : compress_constants(block_range(P.scales, t_r, P.nblocks, P.exact_range));
                        e.bcx = c.x; e.bcy = c.y;
                        // the ring was written through the generic proxy; the TMA unit reads it
                        fence_proxy_async_global();
                        fence_proxy_async();
                        mbar_expect_tx_only(&s_full[lane], kWBufBytes);
                        tma_load_2d(buf, &maps.ring, (int)(t.idx << 5), (int)(t.slot << 8), &s_full[lane], pol_ring);
                        e.tma = 1;
                    }
                    s_desc[lane] = e;
                    ++uses;
                    *reinterpret_cast<volatile uint32_t *>(&s_fills[lane]) = uses;
                    mbar_arrive(&s_full[lane]);
                    state = kBusy;
                    progress = true;
                } else if (give_up) {
                    // the buffer becomes an end marker; a copy in flight lands first
                    const uint32_t par = uses & 1u;
                    publish_end();
                    if (t_tma) (void)mbar_wait(&s_full[lane], par);
                    state = kFree;
                    progress = true;
                }
            }
            __syncwarp();
            // ---- 4. no more tasks: every buffer gets one end marker once it is free
            if (finished && owner && state == kFree && !end_sent) { publish_end(); progress = true; }
            const uint32_t active = __ballot_sync(0xFFFFFFFFu, owner && (state != kFree || !end_sent));
            if (finished && active == 0) break;
            if (__any_sync(0xFFFFFFFFu, progress)) {
                idle = 0;
            } else {
                __nanosleep(256);                       // tasks take microseconds: poll a few times per task
                if (++idle > (1u << 22)) {              // about a second without any progress
                    if (lane == 0) { atomicOr(&P.dev->status, THC_STATUS_WAIT_TIMEOUT); atomicExch(&pc->abort, 1u); }
                    break;
                }
            }
        }
    } else {
        // ================================================================ consumer pairs
        const int pair = (warp - 1) >> 1, h = (warp - 1) & 1;
        const int lx = lane & 7;
        const float gf = (float)P.granularity;
        const uint32_t lut_addr = lut_lane_addr<kLut8>(lut, lane);
        uint32_t pair_par = 0;
        for (uint32_t i = (uint32_t)pair;; i += (uint32_t)kWPairs) {
            const int b = (int)(i % (uint32_t)nbuf);
            const uint32_t use = i / (uint32_t)nbuf;   // this is fill number `use` of buffer b
            // A parity wait tells a phase only from its neighbours, and a pair may get here while an
            // earlier fill of the buffer (another pair's task) is still to come: first wait until
            // the producer has published this fill (a count), then for its phase of the barrier,
            // which completes when the tile has landed.
            bool ok = false;
            for (uint32_t it = 0; it < (1u << 24); ++it) {
                if (*reinterpret_cast<volatile uint32_t *>(&s_fills[b]) > use) { ok = true; break; }
                __nanosleep(32);
            }
            if (!ok || !mbar_wait(&s_full[b], use & 1u)) {
                atomicOr(&P.dev->status, THC_STATUS_WAIT_TIMEOUT);
                atomicExch(&pc->abort, 1u);
                break;
            }
            const WarpDesc me = s_desc[b];
            if (me.end) break;
            float4 *tile = reinterpret_cast<float4 *>(smem + (size_t)b * kWBufBytes);
            float4 v[32];
            const bool is_b = me.is_b != 0;
            float4 *half = tile + h * 1024;
            if (!is_b) {
                // ================================ pass A, round 1: half h of tile idx of worker-block (r, wl)
                const uint64_t j_thread = (uint64_t)me.r * B + ((uint64_t)me.idx << kPLog2) + (uint64_t)h * 4096u +
                                          (uint64_t)lane * 128u;
                const uint4 sg = sign_call(j_thread, P.round, keys);
                const uint32_t sw[4] = {sg.x, sg.y, sg.z, sg.w};
                float4 *base = half + lane * 8;
                if (!me.tma) {
                    // ragged end of the gradient: the thread fetches its own 128 coordinates
                    const float *x = static_cast<const float *>(in.p[me.wl]);
#pragma unroll 1
                    for (int m = 0; m < 32; ++m)
                        base[(m >> 3) * 256 + ((m & 7) ^ lx)] = load_f32x4_masked(x, j_thread + 4u * m, P.d);
                }
#pragma unroll
                for (int m = 0; m < 32; ++m) v[m] = base[(m >> 3) * 256 + ((m & 7) ^ lx)];
#pragma unroll
                for (int m = 0; m < 32; ++m) v[m] = stages01(flip4(v[m], sw[m >> 3] >> ((m & 7) * 4)));
                stages32<5>(v, 0);
#pragma unroll
                for (int m = 0; m < 32; ++m) base[(m >> 3) * 256 + ((m & 7) ^ lx)] = v[m];
                __syncwarp();
            }
            // ================================ round 2 of pass A and round 1 of pass B: one piece of code.
            // The thread's chunk m sits at row0 + m, slot (m & 7) ^ lx: pass A rows 32 (lane >> 3) of its
            // half, pass B rows (t5, t6) = (lane >> 3) & 3 and t7 = h of the panel.
            {
                float4 *base = is_b ? tile + ((((lane >> 3) & 3) << 5) | (h << 7)) * 8 : half + (lane >> 3) * 256;
#pragma unroll
                for (int m = 0; m < 32; ++m) v[m] = base[m * 8 + ((m & 7) ^ lx)];
                stages32<5>(v, 0);
                if (!is_b) {
                    float4 *ring = reinterpret_cast<float4 *>(P.ring + (size_t)me.slot * B + ((size_t)me.idx << kPLog2)) +
                                   h * 1024 + lane;
#pragma unroll
                    for (int m = 0; m < 32; ++m) ring[m * 32] = v[m];
                } else {
#pragma unroll
                    for (int m = 0; m < 32; ++m) base[m * 8 + ((m & 7) ^ lx)] = v[m];
                }
            }
            if (is_b) {
                // ================================ pass B: panel idx of worker-block (r, wl)
                // both warps have written round 1 (a bounded wait, like every other one)
                __syncwarp();
                if (lane == 0) mbar_arrive(&s_pair[pair]);
                if (!mbar_wait(&s_pair[pair], pair_par)) {
                    atomicOr(&P.dev->status, THC_STATUS_WAIT_TIMEOUT);
                    atomicExch(&pc->abort, 1u);
                    break;
                }
                pair_par ^= 1u;
                float4 *base2 = tile + lane * 8;
#pragma unroll
                for (int k2 = 0; k2 < 32; ++k2)
                    v[k2] = base2[(k2 >> 2) * 256 + (((h << 2) | (k2 & 3)) ^ lx)];
                stages32<3>(v, 2);
                // back to the thread's own slots, scaled: the epilogue below is a compact loop
                // over the eight rows (an epilogue unrolled over the 16 units does not fit the
                // instruction cache)
#pragma unroll
                for (int k2 = 0; k2 < 32; ++k2)
                    base2[(k2 >> 2) * 256 + (((h << 2) | (k2 & 3)) ^ lx)] = scale4(v[k2], P.c_block);
                const uint64_t j_lane = (uint64_t)me.r * B + (uint64_t)lane * 4096u + ((uint64_t)me.idx << 5) + (uint64_t)h * 16u;
                unsigned char *pk = static_cast<unsigned char *>(outp.p[me.wl]);
                float *rot = static_cast<float *>(rotated.p[me.wl]);
                const uint32_t worker = P.worker_base + me.wl;
                const float4 *slot0 = base2 + (((h << 2) | 0) ^ lx), *slot1 = base2 + (((h << 2) | 1) ^ lx);
                const float4 *slot2 = base2 + (((h << 2) | 2) ^ lx), *slot3 = base2 + (((h << 2) | 3) ^ lx);
#pragma unroll 1
                for (int t567 = 0; t567 < 8; ++t567) {
                    const uint64_t j = j_lane + (uint64_t)t567 * (32u * 4096u);
                    const float4 r4[4] = {slot0[t567 * 256], slot1[t567 * 256], slot2[t567 * 256], slot3[t567 * 256]};
                    uint64_t zz[2];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const float4 ra = r4[2 * u], rb = r4[2 * u + 1];
                        if (rot != nullptr) {
                            *reinterpret_cast<float4 *>(rot + j + 8 * u) = ra;
                            *reinterpret_cast<float4 *>(rot + j + 8 * u + 4) = rb;
                        }
                        const float rr[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
                        const uint4 rnd = round_call(j + 8 * u, worker, P.round, keys);
                        zz[u] = quantize8<BITS, IDENTITY>(rr, me.bcx, me.bcy, gf, rnd, lut_addr);
                    }
                    store_packed_pair<BITS>(pk, j, zz[0], zz[1]);
                }
            }
            // Finished: the warp's accesses to the buffer are ordered before the TMA unit's next
            // write to it, its stores before the completion the producer will signal.
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_done[b]);
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
